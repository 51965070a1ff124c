// Offline weight preparation: symmetric uniform quantisation, one step size per output
// channel (Section 3.2 Eq. 6; Section 3.3 "Offline Weight Preparation").
//
// One CTA per output channel (row of [N][K]).  The row (<= 34 KB) is read twice: once for
// the absolute maximum, once to quantise; the second read hits L1/L2.  HBM-bound: 2 B read
// + 1 B written per element.  IEEE division and round-half-to-even, no fast-math: the
// result is bit-exact with the definition.
#include "common.cuh"

namespace quasar {

namespace {

constexpr int kQuantThreads = 256;

__global__ void __launch_bounds__(kQuantThreads)
quantize_rows_kernel(const __nv_bfloat16* __restrict__ w, int64_t K, int8_t* __restrict__ q, float* __restrict__ delta) {
  const int64_t n = blockIdx.x;
  const __nv_bfloat16* row = w + n * K;
  int8_t* qrow = q + n * K;
  const int nvec = (int)(K / 8);

  float amax = 0.f;
  for (int v = threadIdx.x; v < nvec; v += kQuantThreads) {
    uint4 u = __ldg(reinterpret_cast<const uint4*>(row) + v);
    const __nv_bfloat162* h = reinterpret_cast<const __nv_bfloat162*>(&u);
#pragma unroll
    for (int i = 0; i < 4; ++i) {
      float2 f = __bfloat1622float2(h[i]);
      amax = fmaxf(amax, fmaxf(fabsf(f.x), fabsf(f.y)));
    }
  }
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) amax = fmaxf(amax, __shfl_xor_sync(0xffffffffu, amax, o));
  __shared__ float s_max[kQuantThreads / 32];
  if ((threadIdx.x & 31) == 0) s_max[threadIdx.x >> 5] = amax;
  __syncthreads();
  amax = s_max[0];
#pragma unroll
  for (int i = 1; i < kQuantThreads / 32; ++i) amax = fmaxf(amax, s_max[i]);

  const float d = (amax == 0.f) ? 1.0f : __fdiv_rn(amax, 127.0f);
  if (threadIdx.x == 0) delta[n] = d;

  for (int v = threadIdx.x; v < nvec; v += kQuantThreads) {
    uint4 u = __ldg(reinterpret_cast<const uint4*>(row) + v);
    const __nv_bfloat162* h = reinterpret_cast<const __nv_bfloat162*>(&u);
    uint32_t out[2];
#pragma unroll
    for (int i = 0; i < 2; ++i) {
      float2 a = __bfloat1622float2(h[2 * i]);
      float2 b = __bfloat1622float2(h[2 * i + 1]);
      int q0 = max(-127, min(127, __float2int_rn(__fdiv_rn(a.x, d))));
      int q1 = max(-127, min(127, __float2int_rn(__fdiv_rn(a.y, d))));
      int q2 = max(-127, min(127, __float2int_rn(__fdiv_rn(b.x, d))));
      int q3 = max(-127, min(127, __float2int_rn(__fdiv_rn(b.y, d))));
      out[i] = (uint32_t)(q0 & 0xff) | ((uint32_t)(q1 & 0xff) << 8) | ((uint32_t)(q2 & 0xff) << 16) |
               ((uint32_t)(q3 & 0xff) << 24);
    }
    reinterpret_cast<uint2*>(qrow)[v] = make_uint2(out[0], out[1]);
  }
}

}  // namespace

int launch_quantize(const __nv_bfloat16* w, int64_t N, int64_t K, int8_t* q, float* delta, cudaStream_t stream) {
  if (N == 0) return QUASAR_OK;
  quantize_rows_kernel<<<(unsigned)N, kQuantThreads, 0, stream>>>(w, K, q, delta);
  QUASAR_LAUNCH_CHECK();
  return QUASAR_OK;
}

}  // namespace quasar
