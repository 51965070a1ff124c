// Stochastic acceptance of a drafted chain (Section 3.1 Eq. 2-3; Section 3.3 "Lossless Rejection
// Sampling"), on the logits the verification pass produced.  Per draft position: target probability
// p = softmax(logits / T) of the drafted token against the drafter's q, accepted while r < min(1, p / q)
// (Eq. 2); at the first rejection a corrective token is drawn from norm(max(0, p - q)) (Eq. 3); if every
// draft is accepted one more token is drawn from the target distribution of the last row.  Random numbers
// are inputs (r_accept per draft position, r_sample per sequence); a token is drawn from unnormalised
// weights by inversion: the smallest v with w_0 + ... + w_v > r_sample * sum(w).  A drafter that gives no
// distribution is the point mass on its token (a retrieval drafter proposes one token with certainty).
//
// Three small kernels, all reductions in a fixed order (results repeat bit for bit): row statistics of the
// softmax (one CTA per block row; HBM-bound: the logits are read once), the accept walk (one thread per
// sequence), the draw (one CTA per sequence: per-thread segment sums, a block scan, a rescan of one segment).
#include <math.h>

#include "common.cuh"

namespace quasar {

namespace {

constexpr int kStatThreads = 512;
constexpr int kDrawThreads = 1024;

struct RowStat {
  float max, sum, p_tok, q_tok;   // softmax statistics of the row; target and draft probability of the next block token
};

__device__ __forceinline__ float block_reduce_max(float v, float* sh) {
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) v = fmaxf(v, __shfl_xor_sync(0xffffffffu, v, o));
  if ((threadIdx.x & 31) == 0) sh[threadIdx.x >> 5] = v;
  __syncthreads();
  float r = sh[0];
  for (int i = 1; i < (int)(blockDim.x >> 5); ++i) r = fmaxf(r, sh[i]);
  __syncthreads();
  return r;
}
__device__ __forceinline__ float block_reduce_sum(float v, float* sh) {
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
  if ((threadIdx.x & 31) == 0) sh[threadIdx.x >> 5] = v;
  __syncthreads();
  float r = 0.f;
  for (int i = 0; i < (int)(blockDim.x >> 5); ++i) r += sh[i];   // warps in order
  __syncthreads();
  return r;
}

__global__ void __launch_bounds__(kStatThreads)
softmax_stats_kernel(const float* __restrict__ logits, const int32_t* __restrict__ tokens, const int32_t* __restrict__ block_len,
                     const float* __restrict__ q_probs, int T_max, int V, float inv_t, RowStat* __restrict__ stats) {
  __shared__ float sh[kStatThreads / 32];
  const int i = blockIdx.x, b = blockIdx.y;
  const int T = block_len[b];
  if (i >= T) return;
  const float* row = logits + ((size_t)b * T_max + i) * V;
  float m = -INFINITY;
  for (int v = threadIdx.x; v < V; v += kStatThreads) m = fmaxf(m, row[v]);
  m = block_reduce_max(m, sh);
  float s = 0.f;
  for (int v = threadIdx.x; v < V; v += kStatThreads) s += expf((row[v] - m) * inv_t);
  s = block_reduce_sum(s, sh);
  if (threadIdx.x == 0) {
    RowStat st{m, s, 0.f, 1.f};
    if (i + 1 < T) {
      const int tok = tokens[b * T_max + i + 1];
      if (tok >= 0 && tok < V) {
        st.p_tok = expf((row[tok] - m) * inv_t) / s;
        if (q_probs != nullptr) st.q_tok = q_probs[((size_t)b * T_max + i) * V + tok];
      } else {
        st.q_tok = 0.f;   // a token outside the vocabulary can only be rejected
      }
    }
    stats[b * T_max + i] = st;
  }
}

// Eq. 2 along the chain; leaves the row to draw from and whether it is the residual of a rejection.
__global__ void accept_walk_kernel(const RowStat* __restrict__ stats, const int32_t* __restrict__ block_len,
                                   const float* __restrict__ r_accept, int B, int T_max, int32_t* __restrict__ accept_len,
                                   int32_t* __restrict__ draw_row, int32_t* __restrict__ draw_residual) {
  const int b = blockIdx.x * blockDim.x + threadIdx.x;
  if (b >= B) return;
  const int T = block_len[b];
  int n = 0, rejected = 0;
  for (int i = 0; i + 1 < T; ++i) {
    const RowStat st = stats[b * T_max + i];
    const float ratio = st.q_tok > 0.f ? fminf(1.f, st.p_tok / st.q_tok) : 0.f;
    if (!(st.q_tok > 0.f) || !(r_accept[b * T_max + i] < ratio)) { rejected = 1; break; }
    ++n;
  }
  accept_len[b] = n;
  draw_row[b] = rejected ? n : T - 1;
  draw_residual[b] = rejected;
}

__device__ __forceinline__ float draw_weight(const float* row, const float* qrow, int tok, int residual, int v, float m,
                                             float inv_t, float inv_sum) {
  const float p = expf((row[v] - m) * inv_t) * inv_sum;
  if (!residual) return p;
  if (qrow != nullptr) return fmaxf(0.f, p - qrow[v]);   // Eq. 3
  return v == tok ? 0.f : p;                             // point-mass drafter
}

__global__ void __launch_bounds__(kDrawThreads)
draw_kernel(const float* __restrict__ logits, const int32_t* __restrict__ tokens, const float* __restrict__ q_probs,
            const RowStat* __restrict__ stats, const int32_t* __restrict__ draw_row, const int32_t* __restrict__ draw_residual,
            const float* __restrict__ r_sample, int T_max, int V, float inv_t, int32_t* __restrict__ next_token) {
  __shared__ float warp_tot[kDrawThreads / 32];
  __shared__ float s_total;
  __shared__ int s_pick;
  const int b = blockIdx.x;
  const int i = draw_row[b];
  int residual = draw_residual[b];
  const float* row = logits + ((size_t)b * T_max + i) * V;
  const float* qrow = (residual && q_probs != nullptr) ? q_probs + ((size_t)b * T_max + i) * V : nullptr;
  const int tok = residual ? tokens[b * T_max + i + 1] : -1;
  const RowStat st = stats[b * T_max + i];
  const float inv_sum = 1.0f / st.sum;
  const int seg = (V + kDrawThreads - 1) / kDrawThreads;
  const int v0 = min(V, (int)threadIdx.x * seg), v1 = min(V, v0 + seg);
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  if (threadIdx.x == 0) s_pick = -1;

  for (int attempt = 0; attempt < 2; ++attempt) {
    // this thread's segment, then an inclusive scan over the threads (lanes, then warps: a fixed order)
    float local = 0.f;
    for (int v = v0; v < v1; ++v) local += draw_weight(row, qrow, tok, residual, v, st.max, inv_t, inv_sum);
    float incl = local;
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) {
      const float up = __shfl_up_sync(0xffffffffu, incl, o);
      if (lane >= o) incl += up;
    }
    float excl = __shfl_up_sync(0xffffffffu, incl, 1);
    if (lane == 0) excl = 0.f;
    if (lane == 31) warp_tot[warp] = incl;
    __syncthreads();
    float before = 0.f;
    for (int w = 0; w < warp; ++w) before += warp_tot[w];
    if (threadIdx.x == kDrawThreads - 1) s_total = before + incl;
    __syncthreads();
    const float total = s_total;
    if (total > 0.f) {
      // the threads' intervals [begin, end) tile [0, total) exactly: a thread's end is the next one's begin
      const float target = r_sample[b] * total;
      const float begin = before + excl, end = before + incl;
      int last_pos = -1;
      if (local > 0.f && begin <= target && target < end) {
        // the segment that holds the target: walk it; if rounding leaves no element, its last positive one
        float acc = begin;
        int pick = -1;
        for (int v = v0; v < v1; ++v) {
          const float w = draw_weight(row, qrow, tok, residual, v, st.max, inv_t, inv_sum);
          if (w > 0.f) last_pos = v;
          acc += w;
          if (acc > target && w > 0.f) { pick = v; break; }
        }
        s_pick = pick >= 0 ? pick : last_pos;
      }
      __syncthreads();
      if (s_pick < 0) {   // r_sample * total rounded up to the total: the last token with a positive weight
        for (int v = v1 - 1; v >= v0 && last_pos < 0; --v)
          if (draw_weight(row, qrow, tok, residual, v, st.max, inv_t, inv_sum) > 0.f) last_pos = v;
        if (last_pos >= 0) atomicMax(&s_pick, last_pos);
        __syncthreads();
      }
      break;
    }
    // max(0, p - q) is empty (p == q): the corrective token comes from p itself
    __syncthreads();
    residual = 0;
    qrow = nullptr;
  }
  if (threadIdx.x == 0) {
    int pick = s_pick;
    if (pick < 0) pick = 0;
    next_token[b] = pick;
  }
}

size_t align256s(size_t v) { return (v + 255) / 256 * 256; }

}  // namespace

size_t accept_stochastic_workspace_bytes(int B, int T_max) {
  return align256s((size_t)B * T_max * sizeof(RowStat)) + 2 * align256s((size_t)B * sizeof(int32_t));
}

int launch_accept_stochastic(const float* logits, const int32_t* tokens, const int32_t* block_len, const float* q_probs, int B,
                             int T_max, int V, float temperature, const float* r_accept, const float* r_sample,
                             int32_t* accept_len, int32_t* next_token, void* workspace, cudaStream_t stream) {
  unsigned char* ws = reinterpret_cast<unsigned char*>(workspace);
  RowStat* stats = reinterpret_cast<RowStat*>(ws);
  int32_t* draw_row = reinterpret_cast<int32_t*>(ws + align256s((size_t)B * T_max * sizeof(RowStat)));
  int32_t* draw_res = reinterpret_cast<int32_t*>(ws + align256s((size_t)B * T_max * sizeof(RowStat)) + align256s((size_t)B * 4));
  const float inv_t = 1.0f / temperature;
  softmax_stats_kernel<<<dim3(T_max, B), kStatThreads, 0, stream>>>(logits, tokens, block_len, q_probs, T_max, V, inv_t, stats);
  QUASAR_LAUNCH_CHECK();
  accept_walk_kernel<<<(B + 63) / 64, 64, 0, stream>>>(stats, block_len, r_accept, B, T_max, accept_len, draw_row, draw_res);
  QUASAR_LAUNCH_CHECK();
  draw_kernel<<<B, kDrawThreads, 0, stream>>>(logits, tokens, q_probs, stats, draw_row, draw_res, r_sample, T_max, V, inv_t,
                                             next_token);
  QUASAR_LAUNCH_CHECK();
  return QUASAR_OK;
}

}  // namespace quasar
