// 4-bit group-wise weights (Section 6, "Ultra-low Bit Verification": weights of 4 bits or fewer, the first
// item of the paper's outlook).  The quantiser is Q of Section 3.2 Eq. 6 with the range [-7, 7] and one
// step size per output channel and group of 128 consecutive input channels; two codes per byte (the even
// input channel in the low nibble, two's complement).  The linear layer is Eq. 8 with one step per group:
//   Y[m][n] = sum_g delta[n][g] * sum_{k in g} X[m][k] * code[n][k]
// The weight stream is a quarter of the bf16 one (Section 3.4's M * bytes / BW term).
//
// Kernel: a CTA of 4 warps owns 64 output channels x a range of groups.  A lane reads 8 packed bytes (16
// codes) of one weight row per step; a code becomes a bf16 by placing (code + 8) under the exponent of 128
// and subtracting 136 (exact), two codes per instruction.  Shifting by 4 bits pairs code i with code i + 4,
// so the activation rows are staged in shared memory in that order (0,4,1,5,2,6,3,7 within eight) and the
// MMA's operands line up without further moves.  mma.m16n8k16 bf16 with fp32 accumulation per group, folded
// into the running sum with the group's step size.  k-ranges are added in a fixed order by a second kernel.
#include "common.cuh"

namespace quasar {

namespace {

constexpr int kGroup = 128;
constexpr int kW4Threads = 128;
constexpr int kW4BlockN = 64;

__global__ void __launch_bounds__(256)
quantize_int4_kernel(const __nv_bfloat16* __restrict__ w, int64_t K, uint8_t* __restrict__ packed, float* __restrict__ delta) {
  const int64_t n = blockIdx.x;
  const int ngroups = (int)(K / kGroup);
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  for (int g = warp; g < ngroups; g += 8) {
    const uint2 raw = __ldg(reinterpret_cast<const uint2*>(w + n * K + (int64_t)g * kGroup) + lane);   // four bf16
    const __nv_bfloat162* h = reinterpret_cast<const __nv_bfloat162*>(&raw);
    const float2 a = __bfloat1622float2(h[0]), b = __bfloat1622float2(h[1]);
    float amax = fmaxf(fmaxf(fabsf(a.x), fabsf(a.y)), fmaxf(fabsf(b.x), fabsf(b.y)));
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) amax = fmaxf(amax, __shfl_xor_sync(0xffffffffu, amax, o));
    const float d = amax == 0.f ? 1.0f : __fdiv_rn(amax, 7.0f);
    const int q0 = max(-7, min(7, __float2int_rn(__fdiv_rn(a.x, d))));
    const int q1 = max(-7, min(7, __float2int_rn(__fdiv_rn(a.y, d))));
    const int q2 = max(-7, min(7, __float2int_rn(__fdiv_rn(b.x, d))));
    const int q3 = max(-7, min(7, __float2int_rn(__fdiv_rn(b.y, d))));
    const unsigned short out = (unsigned short)((q0 & 0xF) | ((q1 & 0xF) << 4) | ((q2 & 0xF) << 8) | ((q3 & 0xF) << 12));
    reinterpret_cast<unsigned short*>(packed + n * (K / 2) + (int64_t)g * (kGroup / 2))[lane] = out;
    if (lane == 0) delta[n * ngroups + g] = d;
  }
}

struct W4Args {
  const __nv_bfloat16* x;    // [M][K]
  const uint8_t* w;          // [N][K/2]
  const float* delta;        // [N][K/128]
  void* y;
  const __nv_bfloat16* res;
  float* partial;            // [nsplit][NT*8][N]
  int M, N, K, groups_per_split, nsplit, y_is_f32;
};

__device__ __forceinline__ void mma_bf16(float (&c)[4], uint32_t a0, uint32_t a1, uint32_t a2, uint32_t a3, uint32_t b0,
                                         uint32_t b1) {
  asm volatile(
      "mma.sync.aligned.m16n8k16.row.col.f32.bf16.bf16.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%0,%1,%2,%3};\n"
      : "+f"(c[0]), "+f"(c[1]), "+f"(c[2]), "+f"(c[3])
      : "r"(a0), "r"(a1), "r"(a2), "r"(a3), "r"(b0), "r"(b1));
}

// eight packed codes -> four bf16 pairs (code i, code i + 4), i = 0..3
__device__ __forceinline__ void nib8_to_bf16(uint32_t w, uint32_t (&out)[4]) {
  const uint32_t u = w ^ 0x88888888u;                 // code + 8 in every nibble
  const __nv_bfloat162 bias = __floats2bfloat162_rn(136.f, 136.f);
#pragma unroll
  for (int i = 0; i < 4; ++i) {
    const uint32_t v = ((u >> (4 * i)) & 0x000F000Fu) | 0x43004300u;     // bf16 128 + (code + 8)
    const __nv_bfloat162 r = __hsub2(*reinterpret_cast<const __nv_bfloat162*>(&v), bias);
    out[i] = *reinterpret_cast<const uint32_t*>(&r);
  }
}

__device__ __forceinline__ void w4_store(const W4Args& a, float v, int m, int n) {
  const size_t idx = (size_t)m * a.N + n;
  if (a.res != nullptr) v = __bfloat162float(__float2bfloat16_rn(v)) + __bfloat162float(a.res[idx]);
  if (a.y_is_f32) reinterpret_cast<float*>(a.y)[idx] = v;
  else reinterpret_cast<__nv_bfloat16*>(a.y)[idx] = __float2bfloat16_rn(v);
}

template <int NT>
__global__ void __launch_bounds__(kW4Threads) w4_gemm_kernel(W4Args a) {
  // one group (128 input channels) of the activation rows at a time: [NT*8][128] bf16, eight-element blocks
  // permuted to 0,4,1,5,2,6,3,7, 16-byte pieces swizzled by row parity
  __shared__ __align__(16) uint4 xs[NT * 8 * 16];
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31, g = lane >> 2, t = lane & 3;
  const int n0 = blockIdx.x * kW4BlockN + warp * 16;
  const int ngroups = a.K / kGroup;
  const int g_begin = blockIdx.y * a.groups_per_split, g_end = min(ngroups, g_begin + a.groups_per_split);
  const int r0 = min(n0 + g, a.N - 1), r1 = min(n0 + g + 8, a.N - 1);
  const uint8_t* wrow0 = a.w + (size_t)r0 * (a.K / 2);
  const uint8_t* wrow1 = a.w + (size_t)r1 * (a.K / 2);
  float tot[NT][4];
#pragma unroll
  for (int i = 0; i < NT; ++i) tot[i][0] = tot[i][1] = tot[i][2] = tot[i][3] = 0.f;

  for (int gi = g_begin; gi < g_end; ++gi) {
    __syncthreads();
    for (int c = threadIdx.x; c < NT * 8 * 16; c += kW4Threads) {
      const int row = c >> 4, pc = c & 15;
      uint4 v = make_uint4(0, 0, 0, 0);
      if (row < a.M) {
        const uint4 raw = *reinterpret_cast<const uint4*>(a.x + (size_t)row * a.K + (size_t)gi * kGroup + pc * 8);
        // halves e0..e7 -> e0,e4,e1,e5,e2,e6,e3,e7
        v.x = __byte_perm(raw.x, raw.z, 0x5410);
        v.y = __byte_perm(raw.x, raw.z, 0x7632);
        v.z = __byte_perm(raw.y, raw.w, 0x5410);
        v.w = __byte_perm(raw.y, raw.w, 0x7632);
      }
      xs[row * 16 + (pc ^ ((row & 1) << 2))] = v;
    }
    __syncthreads();
    const float d0 = __ldg(a.delta + (size_t)r0 * ngroups + gi), d1 = __ldg(a.delta + (size_t)r1 * ngroups + gi);
    float acc[NT][4];
#pragma unroll
    for (int i = 0; i < NT; ++i) acc[i][0] = acc[i][1] = acc[i][2] = acc[i][3] = 0.f;
#pragma unroll
    for (int s = 0; s < 2; ++s) {                       // a step covers 64 input channels: 16 per lane
      const uint2 wa = __ldg(reinterpret_cast<const uint2*>(wrow0 + (size_t)gi * 64 + s * 32) + t);
      const uint2 wb = __ldg(reinterpret_cast<const uint2*>(wrow1 + (size_t)gi * 64 + s * 32) + t);
      uint32_t a_lo[4], a_hi[4], b_lo[4], b_hi[4];
      nib8_to_bf16(wa.x, a_lo); nib8_to_bf16(wa.y, a_hi);
      nib8_to_bf16(wb.x, b_lo); nib8_to_bf16(wb.y, b_hi);
#pragma unroll
      for (int nt = 0; nt < NT; ++nt) {
        const int row = nt * 8 + g;
        const int pc = s * 8 + t * 2;
        const uint4 x0 = xs[row * 16 + (pc ^ ((row & 1) << 2))];
        const uint4 x1 = xs[row * 16 + ((pc + 1) ^ ((row & 1) << 2))];
        mma_bf16(acc[nt], a_lo[0], b_lo[0], a_lo[1], b_lo[1], x0.x, x0.y);
        mma_bf16(acc[nt], a_lo[2], b_lo[2], a_lo[3], b_lo[3], x0.z, x0.w);
        mma_bf16(acc[nt], a_hi[0], b_hi[0], a_hi[1], b_hi[1], x1.x, x1.y);
        mma_bf16(acc[nt], a_hi[2], b_hi[2], a_hi[3], b_hi[3], x1.z, x1.w);
      }
    }
#pragma unroll
    for (int nt = 0; nt < NT; ++nt) {
      tot[nt][0] = fmaf(acc[nt][0], d0, tot[nt][0]);
      tot[nt][1] = fmaf(acc[nt][1], d0, tot[nt][1]);
      tot[nt][2] = fmaf(acc[nt][2], d1, tot[nt][2]);
      tot[nt][3] = fmaf(acc[nt][3], d1, tot[nt][3]);
    }
  }
#pragma unroll
  for (int nt = 0; nt < NT; ++nt) {
#pragma unroll
    for (int e = 0; e < 4; ++e) {
      const int n = n0 + g + (e >> 1) * 8, m = nt * 8 + 2 * t + (e & 1);
      if (n >= a.N || m >= a.M) continue;
      if (a.nsplit == 1) w4_store(a, tot[nt][e], m, n);
      else __stcg(a.partial + ((size_t)blockIdx.y * (NT * 8) + m) * a.N + n, tot[nt][e]);
    }
  }
}

template <int NT>
__global__ void __launch_bounds__(256) w4_reduce_kernel(W4Args a) {
  const int64_t i = (int64_t)blockIdx.x * 256 + threadIdx.x;
  if (i >= (int64_t)a.M * a.N) return;
  const int m = (int)(i / a.N), n = (int)(i % a.N);
  float s = 0.f;
  for (int k = 0; k < a.nsplit; ++k) s += __ldcg(a.partial + ((size_t)k * (NT * 8) + m) * a.N + n);   // fixed order
  w4_store(a, s, m, n);
}

int plan_w4_split(int64_t N, int64_t K, int* groups_per_split) {
  const int nblocks = (int)((N + kW4BlockN - 1) / kW4BlockN);
  const int ngroups = (int)(K / kGroup);
  int want = (148 * 4 + nblocks - 1) / nblocks;
  want = want < 1 ? 1 : (want > ngroups ? ngroups : want);
  want = want > 32 ? 32 : want;
  const int per = (ngroups + want - 1) / want;
  *groups_per_split = per;
  return (ngroups + per - 1) / per;
}

template <int NT>
int launch_w4_nt(const W4Args& a, cudaStream_t stream) {
  w4_gemm_kernel<NT><<<dim3((a.N + kW4BlockN - 1) / kW4BlockN, a.nsplit), kW4Threads, 0, stream>>>(a);
  QUASAR_LAUNCH_CHECK();
  if (a.nsplit > 1) {
    w4_reduce_kernel<NT><<<(unsigned)(((int64_t)a.M * a.N + 255) / 256), 256, 0, stream>>>(a);
    QUASAR_LAUNCH_CHECK();
  }
  return QUASAR_OK;
}

}  // namespace

int launch_quantize_int4(const __nv_bfloat16* w, int64_t N, int64_t K, uint8_t* packed, float* delta, cudaStream_t stream) {
  if (N == 0) return QUASAR_OK;
  quantize_int4_kernel<<<(unsigned)N, 256, 0, stream>>>(w, K, packed, delta);
  QUASAR_LAUNCH_CHECK();
  return QUASAR_OK;
}

size_t linear_w4_workspace_bytes(int64_t M, int64_t N, int64_t K) {
  int per = 0;
  const int nsplit = plan_w4_split(N, K, &per);
  const size_t mpad = (size_t)(((M < 48 ? M : 48) + 7) / 8) * 8;
  return nsplit > 1 ? (size_t)nsplit * mpad * (size_t)N * sizeof(float) : 16;
}

int launch_linear_w4(const __nv_bfloat16* x, const uint8_t* w, const float* delta, int64_t M, int64_t N, int64_t K, void* y,
                     bool y_is_f32, const __nv_bfloat16* residual, void* workspace, size_t workspace_bytes,
                     cudaStream_t stream) {
  if (M <= 0 || N <= 0 || K <= 0 || (K % kGroup) != 0 || N > 0x7fffffff || K > 0x7fffffff) {
    set_error("linear_w4: unsupported sizes M=%lld N=%lld K=%lld (K must be a multiple of %d)", (long long)M, (long long)N,
              (long long)K, kGroup);
    return QUASAR_ERR_SHAPE;
  }
  if (workspace_bytes < linear_w4_workspace_bytes(M, N, K)) {
    set_error("linear_w4: workspace of %zu bytes, need %zu", workspace_bytes, linear_w4_workspace_bytes(M, N, K));
    return QUASAR_ERR_CAPACITY;
  }
  const size_t ybytes = y_is_f32 ? 4 : 2;
  for (int64_t m0 = 0; m0 < M; m0 += 48) {              // blocks of at most 48 rows per launch
    W4Args a;
    a.M = (int)((M - m0) < 48 ? (M - m0) : 48);
    a.N = (int)N; a.K = (int)K;
    a.x = x + m0 * K; a.w = w; a.delta = delta;
    a.y = reinterpret_cast<unsigned char*>(y) + (size_t)m0 * N * ybytes;
    a.res = residual ? residual + m0 * N : nullptr;
    a.partial = reinterpret_cast<float*>(workspace);
    a.nsplit = plan_w4_split(N, K, &a.groups_per_split);
    a.y_is_f32 = y_is_f32 ? 1 : 0;
    int rc;
    switch ((a.M + 7) / 8) {
      case 1: rc = launch_w4_nt<1>(a, stream); break;
      case 2: rc = launch_w4_nt<2>(a, stream); break;
      case 3: rc = launch_w4_nt<3>(a, stream); break;
      case 4: rc = launch_w4_nt<4>(a, stream); break;
      case 5: rc = launch_w4_nt<5>(a, stream); break;
      default: rc = launch_w4_nt<6>(a, stream); break;
    }
    if (rc != QUASAR_OK) return rc;
  }
  return QUASAR_OK;
}

}  // namespace quasar
