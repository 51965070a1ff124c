// The paper's W8A8 form of the linear layer (Section 3.2 Eq. 4-8, Section 3.3 Eq. 9-10):
//   offline   s_j (Eq. 5), W~ = W diag(s)^-1 (Eq. 4), W_int8 = Q(W~, delta_w) (Eq. 6)
//   online    X_int8 = Q(X * s, delta_x) per token, fused smoothing + quantisation (Eq. 9)
//             Y_int32 = W_int8 x X_int8 on the integer tensor cores (Eq. 8),  Y = Y_int32 * (delta_w * delta_x) (Eq. 10)
// Q(., delta) is the same operator everywhere: delta = absmax / 127 (fp32 IEEE division, 1 for an all-zero
// row), q = clamp(round_half_even(v / delta), -127, 127).  No fast-math on any of these paths: the integer
// codes, and with them the int32 accumulators, are bit-exact with the definition.
//
// Direction of s: Eq. 4 and Eq. 9 multiply the activations by s and divide the weights by it; for that to
// shrink an outlier channel (the stated purpose) s_j = max|W_j|^(1-alpha) / max|X_j|^alpha, the reciprocal
// of the expression printed as Eq. 5 (which is the factor the activations are divided by).
#include "common.cuh"

namespace quasar {

namespace {

constexpr int kQuantThreads = 256;

// ---- Eq. 5: column maxima of W, then the factors ----------------------------------------------------
__global__ void __launch_bounds__(256) colmax_kernel(const __nv_bfloat16* __restrict__ w, int64_t N, int64_t K,
                                                     unsigned* __restrict__ colmax_bits) {
  // block: 256 columns x a strip of 64 rows; non-negative floats order like their bit patterns
  const int64_t k = (int64_t)blockIdx.x * 256 + threadIdx.x;
  if (k >= K) return;
  const int64_t n0 = (int64_t)blockIdx.y * 64;
  const int64_t n1 = n0 + 64 < N ? n0 + 64 : N;
  float m = 0.f;
  for (int64_t n = n0; n < n1; ++n) m = fmaxf(m, fabsf(__bfloat162float(w[n * K + k])));
  atomicMax(colmax_bits + k, __float_as_uint(m));
}

__global__ void smooth_factor_kernel(const float* __restrict__ act_absmax, const unsigned* __restrict__ colmax_bits,
                                     int64_t K, double alpha, float* __restrict__ s) {
  const int64_t k = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
  if (k >= K) return;
  const double a = (double)act_absmax[k], wm = (double)__uint_as_float(colmax_bits[k]);
  float out = 1.0f;
  if (a > 0.0 && wm > 0.0) out = (float)(pow(wm, 1.0 - alpha) / pow(a, alpha));
  s[k] = out;
}

// ---- Q(v, delta) per row, v = w (kPlain), w / s (kDivide: offline weights) or x * s (kMultiply: activations) ----
enum SmoothMode { kPlain = 0, kDivide = 1, kMultiply = 2 };

template <int MODE>
__device__ __forceinline__ float smoothed(float v, float s) {
  if (MODE == kDivide) return __fdiv_rn(v, s);
  if (MODE == kMultiply) return __fmul_rn(v, s);
  return v;
}

template <int MODE>
__global__ void __launch_bounds__(kQuantThreads)
quantize_smoothed_kernel(const __nv_bfloat16* __restrict__ w, const float* __restrict__ s, int64_t K,
                         int8_t* __restrict__ q, float* __restrict__ delta) {
  const int64_t n = blockIdx.x;
  const __nv_bfloat16* row = w + n * K;
  int8_t* qrow = q + n * K;
  const int nvec = (int)(K / 8);

  float amax = 0.f;
  for (int v = threadIdx.x; v < nvec; v += kQuantThreads) {
    const uint4 u = __ldg(reinterpret_cast<const uint4*>(row) + v);
    const __nv_bfloat162* h = reinterpret_cast<const __nv_bfloat162*>(&u);
    float sv[8];
#pragma unroll
    for (int i = 0; i < 8; ++i) sv[i] = MODE == kPlain ? 1.f : __ldg(s + (int64_t)v * 8 + i);
#pragma unroll
    for (int i = 0; i < 4; ++i) {
      const float2 f = __bfloat1622float2(h[i]);
      amax = fmaxf(amax, fmaxf(fabsf(smoothed<MODE>(f.x, sv[2 * i])), fabsf(smoothed<MODE>(f.y, sv[2 * i + 1]))));
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
    const uint4 u = __ldg(reinterpret_cast<const uint4*>(row) + v);
    const __nv_bfloat162* h = reinterpret_cast<const __nv_bfloat162*>(&u);
    uint32_t out[2] = {0u, 0u};
#pragma unroll
    for (int i = 0; i < 8; ++i) {
      const float2 f = __bfloat1622float2(h[i >> 1]);
      const float sv = MODE == kPlain ? 1.f : __ldg(s + (int64_t)v * 8 + i);
      const float val = smoothed<MODE>((i & 1) ? f.y : f.x, sv);
      const int qi = max(-127, min(127, __float2int_rn(__fdiv_rn(val, d))));
      out[i >> 2] |= (uint32_t)(qi & 0xff) << (8 * (i & 3));
    }
    reinterpret_cast<uint2*>(qrow)[v] = make_uint2(out[0], out[1]);
  }
}

// ---- the integer GEMM ---------------------------------------------------------------------------------
// Same work split as the weight-only skinny GEMM: a CTA of 4 warps owns 64 output channels x one k-range,
// the weights are the 16-row operand of mma.m16n8k32 (s8 x s8 -> s32), read once with 128-bit streaming
// loads; the quantised activation rows are the 8-wide operand, staged in shared memory.  The contraction
// index may be permuted freely as long as both operands agree: a lane's 16 contiguous weight bytes of one
// row feed the k-slots of two MMAs and meet the 16 activation bytes at the same offsets.  Partial sums of
// the k-ranges are int32: their reduction by the last CTA to arrive is exact whatever the order.
constexpr int kWarps = 4;
constexpr int kThreads = kWarps * 32;
constexpr int kBlockN = kWarps * 16;
constexpr int kSubK = 1024;      // contraction elements (bytes) staged at a time
constexpr int kMaxSplit = 32;
constexpr size_t kCounterBytes = 64 * 1024;
constexpr int64_t kMaxChannels = (int64_t)(kCounterBytes / sizeof(int)) * kBlockN;

struct A8Args {
  const int8_t* xq;          // [M][K]
  const float* dx;           // [M]
  const int8_t* w;           // [N][K]
  const float* dw;           // [N]
  void* y;                   // [M][N] bf16 or fp32
  const __nv_bfloat16* res;  // [M][N] or nullptr
  int32_t* acc_out;          // [M][N] raw accumulators, or nullptr
  int32_t* partial;          // [nsplit][NT*8][N]
  int* counters;
  int M, N, K, k_per_split, nsplit, y_is_f32;
};

__device__ __forceinline__ void mma_s8(int (&c)[4], uint32_t a0, uint32_t a1, uint32_t a2, uint32_t a3, uint32_t b0,
                                       uint32_t b1) {
  asm volatile(
      "mma.sync.aligned.m16n8k32.row.col.s32.s8.s8.s32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%0,%1,%2,%3};\n"
      : "+r"(c[0]), "+r"(c[1]), "+r"(c[2]), "+r"(c[3])
      : "r"(a0), "r"(a1), "r"(a2), "r"(a3), "r"(b0), "r"(b1));
}

// weights are read once: no L1 allocation, evict-first in L2 (the activations and partial sums are what is read again)
__device__ __forceinline__ uint4 ldg_stream(const void* p) {
  uint4 r;
  uint64_t policy;
  asm volatile("createpolicy.fractional.L2::evict_first.b64 %0, 1.0;\n" : "=l"(policy));
  asm volatile("ld.global.nc.L1::no_allocate.L2::cache_hint.v4.u32 {%0,%1,%2,%3}, [%4], %5;\n"
               : "=r"(r.x), "=r"(r.y), "=r"(r.z), "=r"(r.w)
               : "l"(p), "l"(policy));
  return r;
}

__device__ __forceinline__ void a8_store(const A8Args& a, int acc, int m, int n) {
  const size_t idx = (size_t)m * a.N + n;
  if (a.acc_out != nullptr) a.acc_out[idx] = acc;
  // Eq. 10: Y = Y_int32 * (delta_w * delta_x)
  float v = __fmul_rn((float)acc, __fmul_rn(a.dw[n], a.dx[m]));
  if (a.res != nullptr) v = __bfloat162float(__float2bfloat16_rn(v)) + __bfloat162float(a.res[idx]);
  if (a.y_is_f32) reinterpret_cast<float*>(a.y)[idx] = v;
  else reinterpret_cast<__nv_bfloat16*>(a.y)[idx] = __float2bfloat16_rn(v);
}

template <int NT>
__global__ void __launch_bounds__(kThreads) w8a8_gemm_kernel(A8Args a) {
  extern __shared__ __align__(16) unsigned char smem_raw[];
  uint4* xs = reinterpret_cast<uint4*>(smem_raw);   // [NT*8][kSubK/16] 16-byte pieces, swizzled by row parity
  constexpr int kPieces = kSubK / 16;
  constexpr int kUnroll = 4;
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31, g = lane >> 2, t = lane & 3;
  const int n0 = blockIdx.x * kBlockN + warp * 16;
  const int k_begin = blockIdx.y * a.k_per_split;
  const int k_end = min(a.K, k_begin + a.k_per_split);
  const int r0 = min(n0 + g, a.N - 1), r1 = min(n0 + g + 8, a.N - 1);
  const int8_t* wrow0 = a.w + (size_t)r0 * a.K;
  const int8_t* wrow1 = a.w + (size_t)r1 * a.K;

  int acc[NT][4];
#pragma unroll
  for (int i = 0; i < NT; ++i) acc[i][0] = acc[i][1] = acc[i][2] = acc[i][3] = 0;

  for (int kk = k_begin; kk < k_end; kk += kSubK) {
    __syncthreads();
    for (int c = threadIdx.x; c < NT * 8 * kPieces; c += kThreads) {
      const int row = c / kPieces, pc = c % kPieces;
      const int k = kk + pc * 16;
      uint4 v = make_uint4(0, 0, 0, 0);
      if (row < a.M && k < k_end) v = *reinterpret_cast<const uint4*>(a.xq + (size_t)row * a.K + k);
      xs[row * kPieces + (pc ^ ((row & 1) << 2))] = v;
    }
    __syncthreads();
#pragma unroll 1
    for (int s0 = 0; s0 < kPieces / 4; s0 += kUnroll) {   // a warp step covers 64 contraction bytes
      if (kk + s0 * 64 >= k_end) break;
      uint4 wa[kUnroll], wb[kUnroll];
#pragma unroll
      for (int u = 0; u < kUnroll; ++u) {
        const int k = kk + (s0 + u) * 64 + t * 16;
        if (k < k_end) {
          wa[u] = ldg_stream(wrow0 + k);
          wb[u] = ldg_stream(wrow1 + k);
        } else {
          wa[u] = make_uint4(0, 0, 0, 0);
          wb[u] = make_uint4(0, 0, 0, 0);
        }
      }
#pragma unroll
      for (int u = 0; u < kUnroll; ++u) {
        const int pc = (s0 + u) * 4 + t;
#pragma unroll
        for (int nt = 0; nt < NT; ++nt) {
          const int row = nt * 8 + g;
          const uint4 x0 = xs[row * kPieces + (pc ^ ((row & 1) << 2))];
          mma_s8(acc[nt], wa[u].x, wb[u].x, wa[u].y, wb[u].y, x0.x, x0.y);
          mma_s8(acc[nt], wa[u].z, wb[u].z, wa[u].w, wb[u].w, x0.z, x0.w);
        }
      }
    }
  }

  // acc[nt][0..1]: channel n0+g, rows nt*8+2t, +1;  acc[nt][2..3]: channel n0+g+8.
  if (a.nsplit == 1) {
#pragma unroll
    for (int nt = 0; nt < NT; ++nt) {
#pragma unroll
      for (int e = 0; e < 4; ++e) {
        const int n = n0 + g + (e >> 1) * 8, m = nt * 8 + 2 * t + (e & 1);
        if (n < a.N && m < a.M) a8_store(a, acc[nt][e], m, n);
      }
    }
    return;
  }
  int32_t* mine = a.partial + (size_t)blockIdx.y * (NT * 8) * a.N;
#pragma unroll
  for (int nt = 0; nt < NT; ++nt) {
#pragma unroll
    for (int e = 0; e < 4; ++e) {
      const int n = n0 + g + (e >> 1) * 8, m = nt * 8 + 2 * t + (e & 1);
      if (n < a.N && m < a.M) __stcg(mine + (size_t)m * a.N + n, acc[nt][e]);
    }
  }
  __threadfence();
  __syncthreads();
  __shared__ int s_last;
  if (threadIdx.x == 0) s_last = (atomicAdd(a.counters + blockIdx.x, 1) == a.nsplit - 1);
  __syncthreads();
  if (!s_last) return;
  __threadfence();
  const int nb = blockIdx.x * kBlockN;
  for (int i = threadIdx.x; i < kBlockN * a.M; i += kThreads) {
    const int n = nb + (i % kBlockN), m = i / kBlockN;
    if (n >= a.N) continue;
    int sum = 0;
    for (int s = 0; s < a.nsplit; ++s) sum += __ldcg(a.partial + ((size_t)s * (NT * 8) + m) * a.N + n);
    a8_store(a, sum, m, n);
  }
  if (threadIdx.x == 0) a.counters[blockIdx.x] = 0;   // ready for the next launch on this stream
}

struct SplitPlan {
  int nblocks, nsplit, k_per_split;
};

SplitPlan plan_split(int64_t N, int64_t K) {
  SplitPlan p;
  p.nblocks = (int)((N + kBlockN - 1) / kBlockN);
  const int subs = (int)((K + kSubK - 1) / kSubK);
  int want = (148 * 4 + p.nblocks - 1) / p.nblocks;
  want = want < 1 ? 1 : (want > subs ? subs : want);
  want = want > kMaxSplit ? kMaxSplit : want;
  const int subs_per = (subs + want - 1) / want;
  p.k_per_split = subs_per * kSubK;
  p.nsplit = (subs + subs_per - 1) / subs_per;
  return p;
}

template <int NT>
int launch_nt(const A8Args& a, const SplitPlan& p, cudaStream_t stream) {
  const size_t smem = (size_t)NT * 8 * kSubK;
  static bool configured = false;
  if (smem > 48 * 1024 && !configured) {
    QUASAR_CUDA_CHECK(cudaFuncSetAttribute(w8a8_gemm_kernel<NT>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem));
    configured = true;
  }
  w8a8_gemm_kernel<NT><<<dim3(p.nblocks, p.nsplit), kThreads, smem, stream>>>(a);
  QUASAR_LAUNCH_CHECK();
  return QUASAR_OK;
}

size_t align256(size_t v) { return (v + 255) / 256 * 256; }

}  // namespace

int launch_smoothing_factors(const float* act_absmax, const __nv_bfloat16* w, int64_t N, int64_t K, float alpha,
                             float* s_out, cudaStream_t stream) {
  // the column maxima are gathered in the output array itself (as bit patterns); the factor kernel reads
  // entry k and overwrites it
  unsigned* colmax = reinterpret_cast<unsigned*>(s_out);
  QUASAR_CUDA_CHECK(cudaMemsetAsync(colmax, 0, (size_t)K * sizeof(unsigned), stream));
  colmax_kernel<<<dim3((unsigned)((K + 255) / 256), (unsigned)((N + 63) / 64)), 256, 0, stream>>>(w, N, K, colmax);
  QUASAR_LAUNCH_CHECK();
  smooth_factor_kernel<<<(unsigned)((K + 255) / 256), 256, 0, stream>>>(act_absmax, colmax, K, (double)alpha, s_out);
  QUASAR_LAUNCH_CHECK();
  return QUASAR_OK;
}

int launch_quantize_smoothed(const __nv_bfloat16* v, const float* s, int mode, int64_t rows, int64_t K, int8_t* q,
                             float* delta, cudaStream_t stream) {
  if (rows == 0) return QUASAR_OK;
  if (s == nullptr)
    quantize_smoothed_kernel<kPlain><<<(unsigned)rows, kQuantThreads, 0, stream>>>(v, nullptr, K, q, delta);
  else if (mode == kDivide)
    quantize_smoothed_kernel<kDivide><<<(unsigned)rows, kQuantThreads, 0, stream>>>(v, s, K, q, delta);
  else
    quantize_smoothed_kernel<kMultiply><<<(unsigned)rows, kQuantThreads, 0, stream>>>(v, s, K, q, delta);
  QUASAR_LAUNCH_CHECK();
  return QUASAR_OK;
}

size_t linear_w8a8_workspace_bytes(int64_t M, int64_t N, int64_t K) {
  const SplitPlan p = plan_split(N, K);
  const int64_t rows = M < kMaxRowsPerGemm ? M : kMaxRowsPerGemm;
  const size_t mpad = (size_t)((rows + 7) / 8) * 8;
  size_t partial = p.nsplit > 1 ? (size_t)p.nsplit * mpad * (size_t)N * sizeof(int32_t) : 0;
  const int64_t rows_u = M < 80 ? M : 80;
  if (umma_w8a8_usable(rows_u, N, K)) {
    const size_t pu = umma_w8a8_partial_bytes(rows_u, N, K);
    partial = pu > partial ? pu : partial;
  }
  return kCounterBytes + align256((size_t)M * K) + align256((size_t)M * sizeof(float)) + partial;
}

// where launch_linear_w8a8 keeps the quantised activation rows and their step sizes inside its workspace: a kernel that
// produces the operand may write them there itself and pass x == nullptr
void linear_w8a8_operand_slots(void* workspace, int64_t M, int64_t K, int8_t** xq, float** dx) {
  unsigned char* ws = reinterpret_cast<unsigned char*>(workspace);
  *xq = reinterpret_cast<int8_t*>(ws + kCounterBytes);
  *dx = reinterpret_cast<float*>(ws + kCounterBytes + align256((size_t)M * K));
}

int launch_linear_w8a8(const __nv_bfloat16* x, const float* smooth, const int8_t* w, const float* delta_w, int64_t M,
                       int64_t N, int64_t K, void* y, bool y_is_f32, const __nv_bfloat16* residual, int32_t* acc_out,
                       void* workspace, size_t workspace_bytes, int32_t* status, cudaStream_t stream) {
  if (M <= 0 || N <= 0 || K <= 0 || (K % 16) != 0 || N > kMaxChannels || K > 0x7fffffff) {
    set_error("linear_w8a8: unsupported sizes M=%lld N=%lld K=%lld (K must be a multiple of 16, N at most %lld)",
              (long long)M, (long long)N, (long long)K, (long long)kMaxChannels);
    return QUASAR_ERR_SHAPE;
  }
  if (workspace_bytes < linear_w8a8_workspace_bytes(M, N, K)) {
    set_error("linear_w8a8: workspace of %zu bytes, need %zu", workspace_bytes, linear_w8a8_workspace_bytes(M, N, K));
    return QUASAR_ERR_CAPACITY;
  }
  unsigned char* ws = reinterpret_cast<unsigned char*>(workspace);
  int8_t* xq = reinterpret_cast<int8_t*>(ws + kCounterBytes);
  float* dx = reinterpret_cast<float*>(ws + kCounterBytes + align256((size_t)M * K));
  int32_t* partial = reinterpret_cast<int32_t*>(ws + kCounterBytes + align256((size_t)M * K) + align256((size_t)M * sizeof(float)));
  // Eq. 9: fused smoothing + per-token quantisation of the activations
  if (x != nullptr) {   // (nullptr: the producer of the activations has already written xq and dx)
    const int rc0 = launch_quantize_smoothed(x, smooth, kMultiply, M, K, xq, dx, stream);
    if (rc0 != QUASAR_OK) return rc0;
  }
  const SplitPlan p = plan_split(N, K);
  const size_t ybytes = y_is_f32 ? 4 : 2;
  if (M > 8 && umma_w8a8_usable(M < 80 ? M : 80, N, K)) {
    // blocks of more than 8 rows: the contraction runs on tcgen05 with the accumulator in tensor memory
    for (int64_t m0 = 0; m0 < M; m0 += 80) {
      const int64_t rows = (M - m0) < 80 ? (M - m0) : 80;
      const int rc = launch_umma_w8a8(xq + m0 * K, dx + m0, w, delta_w, rows, N, K,
                                      reinterpret_cast<unsigned char*>(y) + (size_t)m0 * N * ybytes, y_is_f32,
                                      residual ? residual + m0 * N : nullptr, acc_out ? acc_out + m0 * N : nullptr,
                                      reinterpret_cast<int*>(workspace), partial, status, stream);
      if (rc != QUASAR_OK) return rc;
    }
    return QUASAR_OK;
  }
  for (int64_t m0 = 0; m0 < M; m0 += kMaxRowsPerGemm) {
    A8Args a;
    a.M = (int)((M - m0) < kMaxRowsPerGemm ? (M - m0) : kMaxRowsPerGemm);
    a.N = (int)N;
    a.K = (int)K;
    a.xq = xq + m0 * K;
    a.dx = dx + m0;
    a.w = w;
    a.dw = delta_w;
    a.y = reinterpret_cast<unsigned char*>(y) + (size_t)m0 * N * ybytes;
    a.res = residual ? residual + m0 * N : nullptr;
    a.acc_out = acc_out ? acc_out + m0 * N : nullptr;
    a.counters = reinterpret_cast<int*>(workspace);
    a.partial = partial;
    a.k_per_split = p.k_per_split;
    a.nsplit = p.nsplit;
    a.y_is_f32 = y_is_f32 ? 1 : 0;
    int rc;
    switch ((a.M + 7) / 8) {
      case 1: rc = launch_nt<1>(a, p, stream); break;
      case 2: rc = launch_nt<2>(a, p, stream); break;
      case 3: rc = launch_nt<3>(a, p, stream); break;
      case 4: rc = launch_nt<4>(a, p, stream); break;
      case 5: rc = launch_nt<5>(a, p, stream); break;
      case 6: rc = launch_nt<6>(a, p, stream); break;
      case 7: rc = launch_nt<7>(a, p, stream); break;
      case 8: rc = launch_nt<8>(a, p, stream); break;
      default: rc = launch_nt<9>(a, p, stream); break;
    }
    if (rc != QUASAR_OK) return rc;
  }
  return QUASAR_OK;
}

}  // namespace quasar
