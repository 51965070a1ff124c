// Skinny quantised GEMM  Y[m][n] = delta[n] * sum_k X[m][k] * W[n][k]  (Section 3.2 Eq. 8 /
// Section 3.3 Eq. 10, weight-only form): M <= 72 activation rows against an [N][K] int8 (or
// bf16) weight matrix that is read exactly once.  HBM-bound on the weight stream
// (1 B per weight, 2*M flop per byte), so the tensor cores are used only to keep up with it.
//
// Mapping: the weights are the 16-row MMA operand ("A" of mma.m16n8k16, rows = output
// channels), the activation rows are the 8-wide operand, zero-padded to a multiple of 8.
// The contraction index may be permuted freely as long as both operands agree, so each
// thread loads 16 contiguous weight bytes of one row with a single 128-bit load and
// treats them as the k-columns its fragment slots need; the matching activations come
// from a swizzled shared-memory copy of the CTA's k-slice of X.  int8 -> bf16 is exact and
// happens in registers; delta[n] is applied once in the epilogue.
//
// Work split: a CTA of 4 warps owns 64 output channels x one k-range; k-ranges of one
// channel block are reduced in a FIXED order by the last CTA to arrive (fp32 partials in
// the workspace, a self-resetting arrival counter), so results are run-to-run identical.
#include <mutex>

#include "common.cuh"

namespace quasar {

namespace {

constexpr int64_t kRows8UmmaMinBytes = (int64_t)1 << 27;   // weight bytes from which blocks of <= 8 rows take the tcgen05 stream kernel

constexpr int kWarps = 4;
constexpr int kThreads = kWarps * 32;
constexpr int kBlockN = kWarps * 16;  // output channels per CTA
constexpr int kSub = 512;             // contraction elements staged in shared memory at a time (blocks of up to 32 rows)
// Wider blocks stage half as much at a time: the activations of 72 rows would otherwise take 72 KB per CTA
// and leave an SM with three CTAs (12 warps) to hide the weight loads behind.
template <int NT>
__host__ __device__ constexpr int sub_of() { return NT > 4 ? 256 : 512; }
constexpr int kMaxSplit = 32;
// The arrival counters of the split-K reduction take a region of fixed size at the start of the
// workspace, so that calls of different widths can share one workspace: no call's partial sums
// land where another call keeps its counters.
constexpr size_t kCounterBytes = 64 * 1024;
constexpr int64_t kMaxChannels = (int64_t)(kCounterBytes / sizeof(int)) * kBlockN;

struct GemmArgs {
  const __nv_bfloat16* x;   // [M][K]
  const void* w;            // [N][K]
  const float* delta;       // [N] or nullptr
  void* y;                  // [M][N] bf16 or fp32
  const __nv_bfloat16* res; // [M][N] or nullptr
  float* partial;           // [nsplit][NT*8][N]
  int* counters;            // [ceil(N / kBlockN)]
  int M, N, K;
  int k_per_split;          // multiple of kSub
  int nsplit;
  int y_is_f32;
};

__device__ __forceinline__ void mma_bf16(float (&c)[4], uint32_t a0, uint32_t a1, uint32_t a2, uint32_t a3,
                                         uint32_t b0, uint32_t b1) {
  asm volatile(
      "mma.sync.aligned.m16n8k16.row.col.f32.bf16.bf16.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%0,%1,%2,%3};\n"
      : "+f"(c[0]), "+f"(c[1]), "+f"(c[2]), "+f"(c[3])
      : "r"(a0), "r"(a1), "r"(a2), "r"(a3), "r"(b0), "r"(b1));
}

// Four signed bytes -> four bf16 (exact): byte i becomes the low mantissa byte of 2^23, which
// after the +128 bias flip reads 2^23 + (v + 128); subtracting 2^23 + 128 leaves v.
__device__ __forceinline__ void s8x4_to_bf16x4(uint32_t w, uint32_t& lo, uint32_t& hi) {
  const uint32_t u = w ^ 0x80808080u;
  const float f0 = __uint_as_float(__byte_perm(u, 0x4B000000u, 0x7440)) - 8388736.f;
  const float f1 = __uint_as_float(__byte_perm(u, 0x4B000000u, 0x7441)) - 8388736.f;
  const float f2 = __uint_as_float(__byte_perm(u, 0x4B000000u, 0x7442)) - 8388736.f;
  const float f3 = __uint_as_float(__byte_perm(u, 0x4B000000u, 0x7443)) - 8388736.f;
  __nv_bfloat162 p0 = __floats2bfloat162_rn(f0, f1);
  __nv_bfloat162 p1 = __floats2bfloat162_rn(f2, f3);
  lo = *reinterpret_cast<uint32_t*>(&p0);
  hi = *reinterpret_cast<uint32_t*>(&p1);
}

__device__ __forceinline__ uint4 ldg_stream(const void* p) {
  uint4 r;
  asm volatile("ld.global.nc.L1::no_allocate.v4.u32 {%0,%1,%2,%3}, [%4];\n"
               : "=r"(r.x), "=r"(r.y), "=r"(r.z), "=r"(r.w)
               : "l"(p));
  return r;
}

template <bool W_INT8>
__device__ __forceinline__ int swz(int chunk, int row) {
  return W_INT8 ? (chunk ^ (row & 1)) : (chunk ^ ((row & 1) << 2));
}

__device__ __forceinline__ float epilogue_value(float acc, float d, const __nv_bfloat16* res, size_t idx) {
  float v = acc * d;
  if (res != nullptr) {
    v = __bfloat162float(__float2bfloat16_rn(v)) + __bfloat162float(res[idx]);
  }
  return v;
}

template <int NT, bool W_INT8>
__global__ void __launch_bounds__(kThreads) skinny_gemm_kernel(GemmArgs a) {
  extern __shared__ __align__(16) unsigned char smem_raw[];
  constexpr int kSub = sub_of<NT>();
  uint4* xs = reinterpret_cast<uint4*>(smem_raw);  // [NT*8][kSub/8] 16-byte chunks, swizzled
  constexpr int kChunksPerRow = kSub / 8;
  constexpr int kStepK = W_INT8 ? 64 : 32;  // contraction elements one warp step covers
  constexpr int kSteps = kSub / kStepK;
  constexpr int kUnroll = 4;

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int g = lane >> 2, t = lane & 3;
  const int n0 = blockIdx.x * kBlockN + warp * 16;
  const int split = blockIdx.y;
  const int k_begin = split * a.k_per_split;
  const int k_end = min(a.K, k_begin + a.k_per_split);

  const int r0 = min(n0 + g, a.N - 1), r1 = min(n0 + g + 8, a.N - 1);
  const size_t wbytes = W_INT8 ? 1 : 2;
  const unsigned char* wrow0 = reinterpret_cast<const unsigned char*>(a.w) + (size_t)r0 * a.K * wbytes;
  const unsigned char* wrow1 = reinterpret_cast<const unsigned char*>(a.w) + (size_t)r1 * a.K * wbytes;

  float acc[NT][4];
#pragma unroll
  for (int i = 0; i < NT; ++i) acc[i][0] = acc[i][1] = acc[i][2] = acc[i][3] = 0.f;

  for (int kk = k_begin; kk < k_end; kk += kSub) {
    __syncthreads();
    // stage X[:, kk : kk + kSub) (zero beyond M or K)
    for (int c = threadIdx.x; c < NT * 8 * kChunksPerRow; c += kThreads) {
      const int row = c / kChunksPerRow, ch = c % kChunksPerRow;
      const int k = kk + ch * 8;
      uint4 v = make_uint4(0, 0, 0, 0);
      if (row < a.M && k < k_end) v = *reinterpret_cast<const uint4*>(a.x + (size_t)row * a.K + k);
      xs[row * kChunksPerRow + swz<W_INT8>(ch, row)] = v;
    }
    __syncthreads();

#pragma unroll 1
    for (int s0 = 0; s0 < kSteps; s0 += kUnroll) {
      if (kk + s0 * kStepK >= k_end) break;
      uint4 wa[kUnroll], wb[kUnroll];
#pragma unroll
      for (int u = 0; u < kUnroll; ++u) {
        const int k = kk + (s0 + u) * kStepK + t * 16 / (int)wbytes;
        if (k < k_end) {
          wa[u] = ldg_stream(wrow0 + (size_t)k * wbytes);
          wb[u] = ldg_stream(wrow1 + (size_t)k * wbytes);
        } else {
          wa[u] = make_uint4(0, 0, 0, 0);
          wb[u] = make_uint4(0, 0, 0, 0);
        }
      }
#pragma unroll
      for (int u = 0; u < kUnroll; ++u) {
        const int s = s0 + u;
        if (W_INT8) {
          uint32_t A0[4], A1[4], A2[4], A3[4];
          const uint32_t* pa = reinterpret_cast<const uint32_t*>(&wa[u]);
          const uint32_t* pb = reinterpret_cast<const uint32_t*>(&wb[u]);
#pragma unroll
          for (int j = 0; j < 4; ++j) {
            s8x4_to_bf16x4(pa[j], A0[j], A2[j]);
            s8x4_to_bf16x4(pb[j], A1[j], A3[j]);
          }
#pragma unroll
          for (int nt = 0; nt < NT; ++nt) {
            const int row = nt * 8 + g;
            const int ch = s * 8 + t * 2;
            const uint4 x0 = xs[row * kChunksPerRow + swz<true>(ch, row)];
            const uint4 x1 = xs[row * kChunksPerRow + swz<true>(ch + 1, row)];
            mma_bf16(acc[nt], A0[0], A1[0], A2[0], A3[0], x0.x, x0.y);
            mma_bf16(acc[nt], A0[1], A1[1], A2[1], A3[1], x0.z, x0.w);
            mma_bf16(acc[nt], A0[2], A1[2], A2[2], A3[2], x1.x, x1.y);
            mma_bf16(acc[nt], A0[3], A1[3], A2[3], A3[3], x1.z, x1.w);
          }
        } else {
#pragma unroll
          for (int nt = 0; nt < NT; ++nt) {
            const int row = nt * 8 + g;
            const int ch = s * 4 + t;
            const uint4 x0 = xs[row * kChunksPerRow + swz<false>(ch, row)];
            mma_bf16(acc[nt], wa[u].x, wb[u].x, wa[u].y, wb[u].y, x0.x, x0.y);
            mma_bf16(acc[nt], wa[u].z, wb[u].z, wa[u].w, wb[u].w, x0.z, x0.w);
          }
        }
      }
    }
  }

  // ---- epilogue ------------------------------------------------------------------------
  // acc[nt][0..1]: channel n0+g, rows nt*8+2t, +1;  acc[nt][2..3]: channel n0+g+8.
  if (a.nsplit == 1) {
#pragma unroll
    for (int nt = 0; nt < NT; ++nt) {
#pragma unroll
      for (int e = 0; e < 4; ++e) {
        const int n = n0 + g + (e >> 1) * 8;
        const int m = nt * 8 + 2 * t + (e & 1);
        if (n < a.N && m < a.M) {
          const float d = a.delta ? a.delta[n] : 1.0f;
          const size_t idx = (size_t)m * a.N + n;
          const float v = epilogue_value(acc[nt][e], d, a.res, idx);
          if (a.y_is_f32) reinterpret_cast<float*>(a.y)[idx] = v;
          else reinterpret_cast<__nv_bfloat16*>(a.y)[idx] = __float2bfloat16_rn(v);
        }
      }
    }
    return;
  }

  float* mine = a.partial + (size_t)split * (NT * 8) * a.N;
#pragma unroll
  for (int nt = 0; nt < NT; ++nt) {
#pragma unroll
    for (int e = 0; e < 4; ++e) {
      const int n = n0 + g + (e >> 1) * 8;
      const int m = nt * 8 + 2 * t + (e & 1);
      if (n < a.N && m < a.M) __stcg(mine + (size_t)m * a.N + n, acc[nt][e]);
    }
  }
  __threadfence();
  __syncthreads();
  __shared__ int s_last;
  if (threadIdx.x == 0) {
    const int prev = atomicAdd(a.counters + blockIdx.x, 1);
    s_last = (prev == a.nsplit - 1);
  }
  __syncthreads();
  if (!s_last) return;
  __threadfence();
  const int nb = blockIdx.x * kBlockN;
  for (int i = threadIdx.x; i < kBlockN * a.M; i += kThreads) {
    const int n = nb + (i % kBlockN), m = i / kBlockN;
    if (n >= a.N) continue;
    float sum = 0.f;
    for (int s = 0; s < a.nsplit; ++s) sum += __ldcg(a.partial + ((size_t)s * (NT * 8) + m) * a.N + n);
    const float d = a.delta ? a.delta[n] : 1.0f;
    const size_t idx = (size_t)m * a.N + n;
    const float v = epilogue_value(sum, d, a.res, idx);
    if (a.y_is_f32) reinterpret_cast<float*>(a.y)[idx] = v;
    else reinterpret_cast<__nv_bfloat16*>(a.y)[idx] = __float2bfloat16_rn(v);
  }
  if (threadIdx.x == 0) a.counters[blockIdx.x] = 0;  // ready for the next launch on this stream
}

struct SplitPlan {
  int nblocks, nsplit, k_per_split;
};

SplitPlan plan_split(int64_t N, int64_t K) {
  SplitPlan p;
  p.nblocks = (int)((N + kBlockN - 1) / kBlockN);
  const int subs = (int)((K + kSub - 1) / kSub);
  const int target = 148 * 4;  // four 4-warp CTAs per SM in flight
  int want = (target + p.nblocks - 1) / p.nblocks;
  want = want < 1 ? 1 : want;
  want = want > subs ? subs : want;
  want = want > kMaxSplit ? kMaxSplit : want;
  const int subs_per = (subs + want - 1) / want;
  p.k_per_split = subs_per * kSub;
  p.nsplit = (subs + subs_per - 1) / subs_per;
  return p;
}

template <int NT, bool W_INT8>
int launch_nt(const GemmArgs& a, const SplitPlan& p, cudaStream_t stream) {
  const size_t smem = (size_t)NT * 8 * sub_of<NT>() * sizeof(__nv_bfloat16);
  static bool configured = false;
  if (smem > 48 * 1024 && !configured) {
    QUASAR_CUDA_CHECK(cudaFuncSetAttribute(skinny_gemm_kernel<NT, W_INT8>,
                                           cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem));
    configured = true;
  }
  dim3 grid(p.nblocks, p.nsplit);
  skinny_gemm_kernel<NT, W_INT8><<<grid, kThreads, smem, stream>>>(a);
  QUASAR_LAUNCH_CHECK();
  return QUASAR_OK;
}

template <bool W_INT8>
int launch_w(const GemmArgs& a, const SplitPlan& p, cudaStream_t stream) {
  const int nt = (a.M + 7) / 8;
  switch (nt) {
    case 1: return launch_nt<1, W_INT8>(a, p, stream);
    case 2: return launch_nt<2, W_INT8>(a, p, stream);
    case 3: return launch_nt<3, W_INT8>(a, p, stream);
    case 4: return launch_nt<4, W_INT8>(a, p, stream);
    case 5: return launch_nt<5, W_INT8>(a, p, stream);
    case 6: return launch_nt<6, W_INT8>(a, p, stream);
    case 7: return launch_nt<7, W_INT8>(a, p, stream);
    case 8: return launch_nt<8, W_INT8>(a, p, stream);
    case 9: return launch_nt<9, W_INT8>(a, p, stream);
    default: set_error("skinny GEMM: %d rows in one launch", a.M); return QUASAR_ERR_SHAPE;
  }
}

}  // namespace

// the least a call needs: without the scratch of the stream kernel that blocks of at most 8 rows take on very large
// matrices WHEN the workspace has room for it (they fall back to the warp-level kernel otherwise)
static size_t linear_workspace_bytes_min(int64_t M, int64_t N, int64_t K) {
  const SplitPlan p = plan_split(N, K);
  const int64_t rows = M < kMaxRowsPerGemm ? M : kMaxRowsPerGemm;
  const size_t mpad = (size_t)((rows + 7) / 8) * 8;
  const size_t counters = kCounterBytes;
  size_t partial = p.nsplit > 1 ? (size_t)p.nsplit * mpad * (size_t)N * sizeof(float) : 0;
  // blocks of more than 8 rows with int8 weights run on the tcgen05 kernel, which keeps an fp16 copy of the
  // activation rows and its own partial sums here
  const int64_t rows_u = M < 80 ? M : 80;
  if (M > 8 && umma_w8a16_usable(rows_u, N, K)) {
    const size_t su = umma_w8a16_scratch_bytes(rows_u, N, K);
    partial = su > partial ? su : partial;
  }
  return counters + partial;
}

static bool rows8_stream_eligible(int64_t M, int64_t N, int64_t K) {
  return M <= 8 && N * K >= kRows8UmmaMinBytes && umma_rows8_usable(M, N, K);
}

size_t linear_workspace_bytes(int64_t M, int64_t N, int64_t K) {
  size_t need = linear_workspace_bytes_min(M, N, K);
  if (rows8_stream_eligible(M, N, K)) {
    const size_t su = kCounterBytes + umma_rows8_scratch_bytes(M, N, K);
    need = su > need ? su : need;
  }
  return need;
}

int launch_linear(const __nv_bfloat16* x, const void* w, const float* delta, int weight_dtype, int64_t M, int64_t N,
                  int64_t K, void* y, bool y_is_f32, const __nv_bfloat16* residual, void* workspace,
                  size_t workspace_bytes, cudaStream_t stream, int32_t* status) {
  if (M <= 0 || N <= 0 || K <= 0 || (K % 16) != 0 || N > kMaxChannels || K > 0x7fffffff) {
    set_error("linear: unsupported sizes M=%lld N=%lld K=%lld (K must be a multiple of 16, N at most %lld)",
              (long long)M, (long long)N, (long long)K, (long long)kMaxChannels);
    return QUASAR_ERR_SHAPE;
  }
  if (workspace_bytes < linear_workspace_bytes_min(M, N, K)) {
    set_error("linear: workspace of %zu bytes, need %zu", workspace_bytes, linear_workspace_bytes(M, N, K));
    return QUASAR_ERR_CAPACITY;
  }
  const SplitPlan p = plan_split(N, K);
  const size_t counters = kCounterBytes;
  const size_t ybytes = y_is_f32 ? 4 : 2;
  if (weight_dtype == QUASAR_W_INT8 && M > 8 && umma_w8a16_usable(M < 80 ? M : 80, N, K)) {
    // a real dense contraction: tcgen05 MMAs with the accumulator in tensor memory (umma_gemm.cu)
    for (int64_t m0 = 0; m0 < M; m0 += 80) {
      const int64_t rows = (M - m0) < 80 ? (M - m0) : 80;
      const int rc = launch_umma_w8a16(x + m0 * K, reinterpret_cast<const int8_t*>(w), delta, rows, N, K,
                                       reinterpret_cast<unsigned char*>(y) + (size_t)m0 * N * ybytes, y_is_f32,
                                       residual ? residual + m0 * N : nullptr,
                                       reinterpret_cast<unsigned char*>(workspace) + counters, status, stream);
      if (rc != QUASAR_OK) return rc;
    }
    return QUASAR_OK;
  }
  // A matrix of LM-head size with at most 8 rows is a long pure stream: the persistent tcgen05 kernel that feeds
  // the int8 tiles straight into integer MMAs (activations as base-256 digits, umma_gemm.cu) sustains a higher
  // rate than the warp-level kernel there; below that size its two extra launches cost more than it gains.
  if (weight_dtype == QUASAR_W_INT8 && rows8_stream_eligible(M, N, K) && workspace_bytes >= kCounterBytes + umma_rows8_scratch_bytes(M, N, K))
    return launch_umma_rows8(x, reinterpret_cast<const int8_t*>(w), delta, M, N, K, y, y_is_f32, residual,
                             reinterpret_cast<unsigned char*>(workspace) + counters, status, stream);
  for (int64_t m0 = 0; m0 < M; m0 += kMaxRowsPerGemm) {
    GemmArgs a;
    a.M = (int)((M - m0) < kMaxRowsPerGemm ? (M - m0) : kMaxRowsPerGemm);
    a.N = (int)N;
    a.K = (int)K;
    a.x = x + m0 * K;
    a.w = w;
    a.delta = weight_dtype == QUASAR_W_INT8 ? delta : nullptr;
    a.y = reinterpret_cast<unsigned char*>(y) + (size_t)m0 * N * ybytes;
    a.res = residual ? residual + m0 * N : nullptr;
    a.counters = reinterpret_cast<int*>(workspace);
    a.partial = reinterpret_cast<float*>(reinterpret_cast<unsigned char*>(workspace) + counters);
    a.k_per_split = p.k_per_split;
    a.nsplit = p.nsplit;
    a.y_is_f32 = y_is_f32 ? 1 : 0;
    const int rc = weight_dtype == QUASAR_W_INT8 ? launch_w<true>(a, p, stream) : launch_w<false>(a, p, stream);
    if (rc != QUASAR_OK) return rc;
  }
  return QUASAR_OK;
}

// ---- the same linear layer with its scratch inside the library ------------------------------------
// Scratch of the split-K reduction for callers that cannot hand over a workspace: a fixed array in
// device memory that every GPU loading the library holds until the process exits.
constexpr size_t kStaticScratchBytes = 4u << 20;
static __device__ __align__(256) unsigned char g_linear_scratch[kStaticScratchBytes];

size_t linear_static_scratch_bytes() { return kStaticScratchBytes; }

int launch_linear_static(const __nv_bfloat16* x, const void* w, const float* delta, int weight_dtype, int64_t M,
                         int64_t N, int64_t K, void* y, bool y_is_f32, const __nv_bfloat16* residual,
                         cudaStream_t stream) {
  if (M <= 0 || N <= 0 || K <= 0 || (K % 16) != 0 || N > kMaxChannels || K > 0x7fffffff) {
    set_error("linear_static: unsupported sizes M=%lld N=%lld K=%lld (K must be a multiple of 16, N at most %lld)",
              (long long)M, (long long)N, (long long)K, (long long)kMaxChannels);
    return QUASAR_ERR_SHAPE;
  }
  const size_t need = linear_workspace_bytes_min(M, N, K);
  if (need > kStaticScratchBytes) {
    set_error("linear_static: M=%lld N=%lld K=%lld needs %zu bytes of scratch, the built-in array holds %zu; "
              "use quasar_linear with a workspace",
              (long long)M, (long long)N, (long long)K, need, kStaticScratchBytes);
    return QUASAR_ERR_CAPACITY;
  }
  // In host code the array's name only stands for the symbol; its device address is looked up once per
  // device (with that device current) and kept.  The lookup comes after the argument checks, so a refused
  // call touches nothing; it is the only step that may make the runtime load the module (and with it
  // materialise the array) - hence "first call outside any capture".
  constexpr int kMaxDevices = 64;
  static void* scratch_of_device[kMaxDevices] = {};
  static std::mutex mu;
  int dev = 0;
  QUASAR_CUDA_CHECK(cudaGetDevice(&dev));
  if (dev < 0 || dev >= kMaxDevices) {
    set_error("linear_static: device ordinal %d not supported (at most %d devices)", dev, kMaxDevices);
    return QUASAR_ERR_CAPACITY;
  }
  void* scratch = nullptr;
  {
    std::lock_guard<std::mutex> lock(mu);
    if (scratch_of_device[dev] == nullptr) {
      void* ptr = nullptr;
      QUASAR_CUDA_CHECK(cudaGetSymbolAddress(&ptr, g_linear_scratch));
      scratch_of_device[dev] = ptr;
    }
    scratch = scratch_of_device[dev];
  }
  // The arrival counters must start at zero; the array keeps whatever the last call left in it.  (Only the
  // split-K form of the warp-level kernel counts arrivals.)
  const bool counts = plan_split(N, K).nsplit > 1 && !(weight_dtype == QUASAR_W_INT8 && M > 8 && umma_w8a16_usable(M < 80 ? M : 80, N, K));
  if (counts) QUASAR_CUDA_CHECK(cudaMemsetAsync(scratch, 0, kCounterBytes, stream));
  return launch_linear(x, w, delta, weight_dtype, M, N, K, y, y_is_f32, residual, scratch, kStaticScratchBytes, stream, nullptr);
}

}  // namespace quasar
