// Drafting by prompt lookup (Section 4.1: the n-gram drafter of all of the paper's experiments; lookup
// range K = (K_min, K_max), Section 4.4 / Table 3).  For n = K_max down to K_min the last n tokens of a
// sequence are looked up in the tokens before them; the most recent earlier occurrence that is followed
// by at least one token wins and the up to gamma tokens that followed it become the draft; the longest n
// with such an occurrence is used.  One CTA per sequence: every thread tests the start positions
// t, t + blockDim, ... for the current n, the largest matching start is taken (an integer maximum: the
// result does not depend on the order of the threads).
#include "common.cuh"

namespace quasar {

namespace {

__global__ void __launch_bounds__(256) ngram_draft_kernel(const int32_t* __restrict__ history, const int32_t* __restrict__ hist_len,
                                                          int S, int gamma, int k_min, int k_max, int32_t* __restrict__ draft,
                                                          int32_t* __restrict__ draft_len) {
  __shared__ int s_best;
  const int b = blockIdx.x;
  const int32_t* h = history + (size_t)b * S;
  const int L = min(max(hist_len[b], 0), S);
  int found_n = 0, found_start = -1;
  for (int n = min(k_max, L - 1); n >= k_min && n >= 1; --n) {
    if (threadIdx.x == 0) s_best = -1;
    __syncthreads();
    int best = -1;
    for (int start = threadIdx.x; start + n <= L - 1; start += blockDim.x) {
      bool same = true;
      for (int j = 0; j < n && same; ++j) same = h[start + j] == h[L - n + j];
      if (same) best = start;                       // starts grow within a thread: the last one is its largest
    }
    if (best >= 0) atomicMax(&s_best, best);
    __syncthreads();
    const int got = s_best;
    __syncthreads();
    if (got >= 0) { found_n = n; found_start = got; break; }
  }
  int len = 0;
  if (found_start >= 0) len = min(gamma, L - (found_start + found_n));
  for (int i = threadIdx.x; i < gamma; i += blockDim.x) draft[(size_t)b * gamma + i] = i < len ? h[found_start + found_n + i] : -1;
  if (threadIdx.x == 0) draft_len[b] = len;
}

}  // namespace

int launch_ngram_draft(const int32_t* history, const int32_t* hist_len, int B, int S, int gamma, int k_min, int k_max,
                       int32_t* draft, int32_t* draft_len, cudaStream_t stream) {
  ngram_draft_kernel<<<B, 256, 0, stream>>>(history, hist_len, S, gamma, k_min, k_max, draft, draft_len);
  QUASAR_LAUNCH_CHECK();
  return QUASAR_OK;
}

}  // namespace quasar
