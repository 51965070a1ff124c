// The quantised linear layer for blocks of 9 to 72 rows on the 5th-generation tensor cores
// (tcgen05.mma with the accumulator in tensor memory): the regime of the batched and tree
// workloads, where  Y = delta * (W X)  (Section 3.2 Eq. 8 / Section 3.3 Eq. 10) is a real dense
// contraction (2 M flop per weight byte, M up to 72) and no longer a pure weight stream.
//
// Mapping.  A CTA owns 128 output channels x one range of the contraction index.  The weights
// are the 128-row operand A (K-major), the activation rows - padded to a multiple of 16 - the
// operand B (K-major); the 128 x Mpad accumulator lives in tensor memory (one lane per output
// channel, one column per activation row) and never touches registers until the epilogue.
//   * W8A8 (kind::i8, s8 x s8 -> s32): tiles of 128 rows x 128 contraction bytes are brought in by
//     TMA (cp.async.bulk.tensor, 128-byte swizzle) exactly as the MMA reads them - no instruction
//     touches a weight byte.  Accumulators are exact integers.
//   * W8A16 (kind::f16, fp16 x fp16 -> f32): the same int8 tiles land in a raw ring; four warps turn each
//     row into fp16 in registers (int8 -> fp16 is exact) and store it into tensor memory, from where the MMA
//     reads operand A - which is what the weight-only form costs on this path: one conversion instruction
//     per two weights and two bytes of tensor-memory stores per weight.
//   * at most 8 rows on a very large matrix: a persistent stream kernel in which the 16-bit activations ride
//     the integer MMAs as three int8 digits (further down).
// Roles: warp 0 issues the TMA loads, warp 1 the MMAs (one elected thread), warps 2-5 convert
// (W8A16) and run the epilogue (tcgen05.ld, one tensor-memory lane = one output channel per
// thread).  k-ranges of one channel block are added up in a fixed order by a second, fully parallel kernel.
//
// Every wait is bounded (2 s): on expiry the CTA raises an error word, stops waiting everywhere,
// releases its tensor memory and returns.
#include <cuda.h>
#include <cudaTypedefs.h>

#include <mutex>

#include "common.cuh"

namespace quasar {

namespace {

constexpr int kTileN = 128;          // output channels per CTA (MMA M)
constexpr int kTileKBytes = 128;     // contraction bytes of int8 per stage (one 128-byte swizzle row)
constexpr int kStagesI8 = 4;         // two CTAs share an SM: one's epilogue overlaps the other's stream
constexpr int kThreadsU = 192;
constexpr int kMaxMpad = 80;
constexpr unsigned long long kBudgetNs = 2000000000ull;
constexpr size_t kCounterBytesU = 64 * 1024;

struct UmmaArgs {
  const float* dx;           // [M] activation step sizes (W8A8) or nullptr
  const float* dw;           // [N]
  void* y;                   // [M][N] bf16 or fp32
  const __nv_bfloat16* res;  // [M][N] or nullptr
  int32_t* acc_out;          // [M][N] raw accumulators (W8A8) or nullptr
  void* partial;             // [nsplit][Mpad][N] 32-bit words
  int* counters;
  int32_t* error;            // device status word (or nullptr): QUASAR_ERR_TIMEOUT when a wait ran out
  int M, Mpad, N, K, k_per_split, nsplit, y_is_f32;
  int direct;                // 1: one k-range and the kernel itself applies the epilogue; 0: 32-bit partial sums go to `partial`
};

__device__ __forceinline__ uint32_t smem_u32(const void* p) { return (uint32_t)__cvta_generic_to_shared(p); }
__device__ __forceinline__ unsigned long long gtime_ns() {
  unsigned long long t;
  asm volatile("mov.u64 %0, %%globaltimer;\n" : "=l"(t));
  return t;
}
__device__ __forceinline__ void mbar_init(uint64_t* bar, int count) {
  asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;\n" ::"r"(smem_u32(bar)), "r"(count) : "memory");
}
__device__ __forceinline__ void mbar_expect_tx(uint64_t* bar, uint32_t bytes) {
  asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;\n" ::"r"(smem_u32(bar)), "r"(bytes) : "memory");
}
__device__ __forceinline__ void mbar_arrive(uint64_t* bar) {
  asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];\n" ::"r"(smem_u32(bar)) : "memory");
}
__device__ __forceinline__ bool mbar_try(uint64_t* bar, uint32_t parity) {
  uint32_t ok;
  asm volatile("{\n.reg .pred p;\nmbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\nselp.u32 %0, 1, 0, p;\n}\n"
               : "=r"(ok)
               : "r"(smem_u32(bar)), "r"(parity)
               : "memory");
  return ok != 0;
}
// bounded wait; false when it ran out or another thread of the CTA already gave up
__device__ __noinline__ bool mbar_wait(uint64_t* bar, uint32_t parity, volatile int* abort_flag, int32_t* error) {
  if (mbar_try(bar, parity)) return true;
  const unsigned long long t0 = gtime_ns();
  unsigned it = 0;
  while (!mbar_try(bar, parity)) {
    if ((++it & 63u) == 0) {
      if (*abort_flag) return false;
      if (gtime_ns() - t0 > kBudgetNs) {
        *abort_flag = 1;
        if (error != nullptr) atomicMin(error, QUASAR_ERR_TIMEOUT);
        return false;
      }
    }
  }
  return true;
}

__device__ __forceinline__ void tma_load_2d(void* smem_dst, const CUtensorMap* map, int x, int y, uint64_t* bar) {
  asm volatile(
      "cp.async.bulk.tensor.2d.shared::cluster.global.tile.mbarrier::complete_tx::bytes [%0], [%1, {%3, %4}], [%2];\n" ::"r"(
          smem_u32(smem_dst)),
      "l"(map), "r"(smem_u32(bar)), "r"(x), "r"(y)
      : "memory");
}

// The same for a tile that is read once (weights): evict-first in L2, so that the stream does not push out the activation
// rows and partial sums that are read again.
__device__ __forceinline__ uint64_t l2_evict_first_policy() {
  uint64_t policy;
  asm volatile("createpolicy.fractional.L2::evict_first.b64 %0, 1.0;\n" : "=l"(policy));
  return policy;
}
__device__ __forceinline__ void tma_load_2d_stream(void* smem_dst, const CUtensorMap* map, int x, int y, uint64_t* bar, uint64_t policy) {
  asm volatile(
      "cp.async.bulk.tensor.2d.shared::cluster.global.tile.mbarrier::complete_tx::bytes.L2::cache_hint [%0], [%1, {%3, %4}], [%2], %5;\n" ::"r"(
          smem_u32(smem_dst)),
      "l"(map), "r"(smem_u32(bar)), "r"(x), "r"(y), "l"(policy)
      : "memory");
}

// K-major operand tile with 128-byte swizzle: rows of 128 bytes, groups of 8 rows 1024 bytes apart.
__device__ __forceinline__ uint64_t umma_desc_sw128(const void* smem_tile) {
  uint64_t d = 0;
  d |= (uint64_t)((smem_u32(smem_tile) & 0x3ffff) >> 4);   // start address, 16-byte units
  d |= (uint64_t)1 << 16;                                  // leading-dimension offset: unused with this swizzle
  d |= (uint64_t)(1024 >> 4) << 32;                        // stride between 8-row groups
  d |= (uint64_t)1 << 46;                                  // descriptor version of this architecture
  d |= (uint64_t)2 << 61;                                  // 128-byte swizzle
  return d;
}

// instruction descriptor: dense, A and B K-major, M = 128, N = n
__device__ __forceinline__ uint32_t umma_idesc(int c_format, int ab_format, int n) {
  return ((uint32_t)c_format << 4) | ((uint32_t)ab_format << 7) | ((uint32_t)ab_format << 10) | ((uint32_t)(n >> 3) << 17) |
         ((uint32_t)(kTileN >> 4) << 24);
}

template <bool I8>
__device__ __forceinline__ void umma_ss(uint32_t tmem_d, uint64_t desc_a, uint64_t desc_b, uint32_t idesc, uint32_t accumulate) {
  if (I8) {
    asm volatile(
        "{\n.reg .pred p;\nsetp.ne.b32 p, %4, 0;\n"
        "tcgen05.mma.cta_group::1.kind::i8 [%0], %1, %2, %3, p;\n}\n" ::"r"(tmem_d),
        "l"(desc_a), "l"(desc_b), "r"(idesc), "r"(accumulate)
        : "memory");
  } else {
    asm volatile(
        "{\n.reg .pred p;\nsetp.ne.b32 p, %4, 0;\n"
        "tcgen05.mma.cta_group::1.kind::f16 [%0], %1, %2, %3, p;\n}\n" ::"r"(tmem_d),
        "l"(desc_a), "l"(desc_b), "r"(idesc), "r"(accumulate)
        : "memory");
  }
}
__device__ __forceinline__ void umma_commit(uint64_t* bar) {
  asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];\n" ::"r"(smem_u32(bar)) : "memory");
}

// 16 consecutive accumulator columns of this thread's tensor-memory lane
__device__ __forceinline__ void tmem_ld16(uint32_t taddr, uint32_t (&v)[16]) {
  asm volatile(
      "tcgen05.ld.sync.aligned.32x32b.x16.b32 {%0,%1,%2,%3,%4,%5,%6,%7,%8,%9,%10,%11,%12,%13,%14,%15}, [%16];\n"
      : "=r"(v[0]), "=r"(v[1]), "=r"(v[2]), "=r"(v[3]), "=r"(v[4]), "=r"(v[5]), "=r"(v[6]), "=r"(v[7]), "=r"(v[8]), "=r"(v[9]),
        "=r"(v[10]), "=r"(v[11]), "=r"(v[12]), "=r"(v[13]), "=r"(v[14]), "=r"(v[15])
      : "r"(taddr));
  asm volatile("tcgen05.wait::ld.sync.aligned;\n" ::: "memory");
}

template <bool I8>
__device__ __forceinline__ void store_output(const UmmaArgs& a, uint32_t bits, int m, int n) {
  const size_t idx = (size_t)m * a.N + n;
  float v;
  if (I8) {
    const int acc = (int)bits;
    if (a.acc_out != nullptr) a.acc_out[idx] = acc;
    v = __fmul_rn((float)acc, __fmul_rn(a.dw[n], a.dx[m]));   // Eq. 10
  } else {
    v = (__uint_as_float(bits) * a.dx[m]) * a.dw[n];   // the row's power-of-two scale back out (exact), then the step size
  }
  if (a.res != nullptr) v = __bfloat162float(__float2bfloat16_rn(v)) + __bfloat162float(a.res[idx]);
  if (a.y_is_f32) reinterpret_cast<float*>(a.y)[idx] = v;
  else reinterpret_cast<__nv_bfloat16*>(a.y)[idx] = __float2bfloat16_rn(v);
}

// shared memory of the W8A8 kernel: kStagesI8 x (A tile 16 KB + B tile Mpad x 128 B), then barriers
template <bool I8>
__global__ void __launch_bounds__(kThreadsU, 2)
umma_gemm_kernel(const __grid_constant__ CUtensorMap map_w, const __grid_constant__ CUtensorMap map_x, UmmaArgs a) {
  static_assert(I8, "this entry is the int8 x int8 form");
  extern __shared__ __align__(16) unsigned char smem_raw[];
  // operand tiles start on a 1024-byte boundary (the swizzle pattern repeats every 8 rows of 128 bytes)
  unsigned char* smem = smem_raw + ((1024u - (smem_u32(smem_raw) & 1023u)) & 1023u);
  const int b_bytes = a.Mpad * kTileKBytes;                        // multiple of 1024 (Mpad is a multiple of 16)
  const int stage_bytes = kTileN * kTileKBytes + b_bytes;
  unsigned char* tiles = smem;
  uint64_t* full = reinterpret_cast<uint64_t*>(smem + kStagesI8 * stage_bytes);
  uint64_t* empty = full + kStagesI8;
  uint64_t* accum_done = empty + kStagesI8;
  uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(accum_done + 1);
  volatile int* abort_flag = reinterpret_cast<volatile int*>(tmem_slot + 1);

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int n0 = blockIdx.x * kTileN;
  const int k_begin = blockIdx.y * a.k_per_split;
  const int k_end = min(a.K, k_begin + a.k_per_split);
  const int nkb = (k_end - k_begin + kTileKBytes - 1) / kTileKBytes;

  if (threadIdx.x == 0) {
    *abort_flag = 0;
    for (int s = 0; s < kStagesI8; ++s) {
      mbar_init(full + s, 1);
      mbar_init(empty + s, 1);
    }
    mbar_init(accum_done, 1);
    asm volatile("fence.mbarrier_init.release.cluster;\n" ::: "memory");
  }
  if (warp == 1) {   // 128 columns of tensor memory for the 128 x Mpad accumulator
    asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;\n" ::"r"(smem_u32(tmem_slot)), "r"(128u)
                 : "memory");
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;\n" ::: "memory");
  }
  asm volatile("tcgen05.fence::before_thread_sync;\n" ::: "memory");
  __syncthreads();
  asm volatile("tcgen05.fence::after_thread_sync;\n" ::: "memory");
  const uint32_t tmem_base = *tmem_slot;

  if (warp == 0) {
    if (lane == 0) {   // ---- TMA producer ----
      const uint64_t wpolicy = l2_evict_first_policy();
      int s = 0;
      uint32_t ph = 0;
      for (int kb = 0; kb < nkb; ++kb) {
        if (!mbar_wait(empty + s, ph ^ 1u, abort_flag, a.error)) break;
        unsigned char* at = tiles + s * stage_bytes;
        mbar_expect_tx(full + s, (uint32_t)stage_bytes);
        tma_load_2d_stream(at, &map_w, k_begin + kb * kTileKBytes, n0, full + s, wpolicy);
        tma_load_2d(at + kTileN * kTileKBytes, &map_x, k_begin + kb * kTileKBytes, 0, full + s);
        if (++s == kStagesI8) { s = 0; ph ^= 1u; }
      }
    }
  } else if (warp == 1) {
    if (lane == 0) {   // ---- MMA issuer ----
      const uint32_t idesc = umma_idesc(/*s32*/ 2, /*signed int8*/ 1, a.Mpad);
      int s = 0;
      uint32_t ph = 0;
      bool ok = true;
      for (int kb = 0; kb < nkb && ok; ++kb) {
        if (!(ok = mbar_wait(full + s, ph, abort_flag, a.error))) break;
        asm volatile("tcgen05.fence::after_thread_sync;\n" ::: "memory");
        const unsigned char* at = tiles + s * stage_bytes;
        const uint64_t da = umma_desc_sw128(at), db = umma_desc_sw128(at + kTileN * kTileKBytes);
#pragma unroll
        for (int j = 0; j < kTileKBytes / 32; ++j)   // one instruction contracts 32 bytes of k: 32 bytes further along the row
          umma_ss<true>(tmem_base, da + (uint64_t)(j * 2), db + (uint64_t)(j * 2), idesc, (kb > 0 || j > 0) ? 1u : 0u);
        umma_commit(empty + s);   // arrives when the MMAs above have read the stage
        if (++s == kStagesI8) { s = 0; ph ^= 1u; }
      }
      if (ok) umma_commit(accum_done);
    }
  } else {
    // ---- epilogue: warps 2..5; a warp may touch the tensor-memory lanes 32 (warp % 4) .. + 31 ----
    const int q = warp & 3;
    const int n = n0 + q * 32 + lane;
    int got = 1;
    if (lane == 0) got = mbar_wait(accum_done, 0, abort_flag, a.error) ? 1 : 0;
    got = __shfl_sync(0xffffffffu, got, 0);
    if (got) {
      asm volatile("tcgen05.fence::after_thread_sync;\n" ::: "memory");
      for (int c0 = 0; c0 < a.Mpad; c0 += 16) {
        uint32_t v[16];
        tmem_ld16(tmem_base + ((uint32_t)(q * 32) << 16) + (uint32_t)c0, v);
        if (n < a.N) {
#pragma unroll
          for (int j = 0; j < 16; ++j) {
            const int m = c0 + j;
            if (m >= a.M) continue;
            if (a.direct) store_output<true>(a, v[j], m, n);
            else __stcg(reinterpret_cast<uint32_t*>(a.partial) + ((size_t)blockIdx.y * a.Mpad + m) * a.N + n, v[j]);
          }
        }
      }
    }
  }
  asm volatile("tcgen05.fence::before_thread_sync;\n" ::: "memory");
  __threadfence();
  __syncthreads();
  if (warp == 1) {
    asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;\n" ::"r"(tmem_base), "r"(128u) : "memory");
  }
}

// k-ranges of a channel block meet here: a second, fully parallel kernel adds the partial sums in a fixed
// order (split 0, 1, ...) and applies the epilogue.  One thread per activation row and four channels.
template <bool I8>
__global__ void __launch_bounds__(256) umma_reduce_kernel(UmmaArgs a) {
  const int n4 = (a.N + 3) / 4;
  const int64_t i = (int64_t)blockIdx.x * 256 + threadIdx.x;
  if (i >= (int64_t)a.M * n4) return;
  const int m = (int)(i / n4), n = (int)(i % n4) * 4;
  const uint32_t* p0 = reinterpret_cast<const uint32_t*>(a.partial) + (size_t)m * a.N + n;
  const size_t split_stride = (size_t)a.Mpad * a.N;
  if (n + 4 <= a.N && (a.N & 3) == 0) {
    uint4 v[8];
    int ai[4] = {0, 0, 0, 0};
    float af[4] = {0.f, 0.f, 0.f, 0.f};
    for (int s0 = 0; s0 < a.nsplit; s0 += 8) {
      const int cnt = min(8, a.nsplit - s0);
#pragma unroll
      for (int j = 0; j < 8; ++j)
        if (j < cnt) v[j] = __ldcg(reinterpret_cast<const uint4*>(p0 + (size_t)(s0 + j) * split_stride));
#pragma unroll
      for (int j = 0; j < 8; ++j) {
        if (j >= cnt) continue;
        const uint32_t w[4] = {v[j].x, v[j].y, v[j].z, v[j].w};
#pragma unroll
        for (int e = 0; e < 4; ++e) {
          if (I8) ai[e] += (int)w[e];
          else af[e] += __uint_as_float(w[e]);
        }
      }
    }
#pragma unroll
    for (int e = 0; e < 4; ++e) store_output<I8>(a, I8 ? (uint32_t)ai[e] : __float_as_uint(af[e]), m, n + e);
  } else {
    for (int e = 0; e < 4 && n + e < a.N; ++e) {
      int si = 0;
      float sf = 0.f;
      for (int s = 0; s < a.nsplit; ++s) {
        const uint32_t w = __ldcg(p0 + e + (size_t)s * split_stride);
        if (I8) si += (int)w; else sf += __uint_as_float(w);
      }
      store_output<I8>(a, I8 ? (uint32_t)si : __float_as_uint(sf), m, n + e);
    }
  }
}

// ---- the weight-only form (int8 weights, 16-bit activations) on the same tensor cores -------------------
// kind::f16 takes both operands as fp16.  The activations are turned into fp16 once per call by a
// small pre-pass (exact: a bf16 value times a power of two that puts the row's maximum in [2^14, 2^15) is
// an fp16 value unless it lies 2^-39 below that maximum).  The weights never exist as a 16-bit tile in shared
// memory: operand A of the MMA is read from TENSOR memory.  A stage's 128 rows x 64 contraction bytes land by
// TMA (64-byte swizzle); thread r of the four converter warps turns row r into 64 fp16 values in registers -
// the byte with its sign bit flipped under the high byte 0x64 reads 1024 + (w + 128), one packed subtraction
// of 1152 leaves w - and stores them with one tcgen05.st into lane r of the stage's 32 tensor-memory columns
// (two fp16 per column, contraction index ascending).  Per stage the shared memory holds the raw weights
// (8 KB) and the activations (Mpad x 128 B) only, which is what lets five stages of two CTAs fit an SM: the
// kernel's speed is set by the bytes it keeps in flight.
constexpr int kStagesF16 = 5;
constexpr int kRawBytes = kTileN * 64;          // 8 KB
constexpr int kAColsPerStage = 32;              // 64 fp16 per row
constexpr int kAccCols = 96;                    // accumulator columns (Mpad <= 80), then kStagesF16 x 32 columns of A
constexpr int kTmemColsF16 = 256;

__device__ __forceinline__ void s8x4_to_f16x4(uint32_t w, uint32_t& lo, uint32_t& hi) {
  const uint32_t u = w ^ 0x80808080u;
  const uint32_t l = __byte_perm(u, 0x64646464u, 0x4140);
  const uint32_t h = __byte_perm(u, 0x64646464u, 0x4342);
  const __half2 bias = __halves2half2(__ushort_as_half(0x6480), __ushort_as_half(0x6480));   // 1152
  const __half2 lo2 = __hsub2(*reinterpret_cast<const __half2*>(&l), bias);
  const __half2 hi2 = __hsub2(*reinterpret_cast<const __half2*>(&h), bias);
  lo = *reinterpret_cast<const uint32_t*>(&lo2);
  hi = *reinterpret_cast<const uint32_t*>(&hi2);
}

// 32 consecutive columns of this thread's tensor-memory lane
__device__ __forceinline__ void tmem_st32(uint32_t taddr, const uint32_t (&v)[32]) {
  asm volatile(
      "tcgen05.st.sync.aligned.32x32b.x32.b32 [%0], {%1,%2,%3,%4,%5,%6,%7,%8,%9,%10,%11,%12,%13,%14,%15,%16,%17,%18,%19,%20,"
      "%21,%22,%23,%24,%25,%26,%27,%28,%29,%30,%31,%32};\n" ::"r"(taddr),
      "r"(v[0]), "r"(v[1]), "r"(v[2]), "r"(v[3]), "r"(v[4]), "r"(v[5]), "r"(v[6]), "r"(v[7]), "r"(v[8]), "r"(v[9]), "r"(v[10]),
      "r"(v[11]), "r"(v[12]), "r"(v[13]), "r"(v[14]), "r"(v[15]), "r"(v[16]), "r"(v[17]), "r"(v[18]), "r"(v[19]), "r"(v[20]),
      "r"(v[21]), "r"(v[22]), "r"(v[23]), "r"(v[24]), "r"(v[25]), "r"(v[26]), "r"(v[27]), "r"(v[28]), "r"(v[29]), "r"(v[30]),
      "r"(v[31])
      : "memory");
  asm volatile("tcgen05.wait::st.sync.aligned;\n" ::: "memory");
}

// D[tmem] (+)= A[tmem] * B[smem descriptor], fp16 x fp16 -> fp32
__device__ __forceinline__ void umma_ts_f16(uint32_t tmem_d, uint32_t tmem_a, uint64_t desc_b, uint32_t idesc, uint32_t accumulate) {
  asm volatile(
      "{\n.reg .pred p;\nsetp.ne.b32 p, %4, 0;\n"
      "tcgen05.mma.cta_group::1.kind::f16 [%0], [%1], %2, %3, p;\n}\n" ::"r"(tmem_d),
      "r"(tmem_a), "l"(desc_b), "r"(idesc), "r"(accumulate)
      : "memory");
}

__global__ void __launch_bounds__(kThreadsU, 2)
umma_w8a16_kernel(const __grid_constant__ CUtensorMap map_w, const __grid_constant__ CUtensorMap map_x, UmmaArgs a) {
  extern __shared__ __align__(16) unsigned char smem_raw[];
  unsigned char* smem = smem_raw + ((1024u - (smem_u32(smem_raw) & 1023u)) & 1023u);
  const int b_bytes = a.Mpad * 128;                               // Mpad rows x 64 fp16
  const int stage_bytes = b_bytes + kRawBytes;                    // [activations][raw weights]
  unsigned char* tiles = smem;
  uint64_t* full = reinterpret_cast<uint64_t*>(smem + kStagesF16 * stage_bytes);   // TMA landed (raw weights + activations)
  uint64_t* conv = full + kStagesF16;                                              // fp16 weights stored to tensor memory
  uint64_t* empty = conv + kStagesF16;                                             // MMAs of the stage done
  uint64_t* accum_done = empty + kStagesF16;
  uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(accum_done + 1);
  volatile int* abort_flag = reinterpret_cast<volatile int*>(tmem_slot + 1);

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int n0 = blockIdx.x * kTileN;
  const int k_begin = blockIdx.y * a.k_per_split;
  const int k_end = min(a.K, k_begin + a.k_per_split);
  const int nkb = (k_end - k_begin + 63) / 64;

  if (threadIdx.x == 0) {
    *abort_flag = 0;
    for (int s = 0; s < kStagesF16; ++s) {
      mbar_init(full + s, 1);
      mbar_init(conv + s, 4);     // one arrival per converter warp
      mbar_init(empty + s, 1);
    }
    mbar_init(accum_done, 1);
    asm volatile("fence.mbarrier_init.release.cluster;\n" ::: "memory");
  }
  if (warp == 1) {
    asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;\n" ::"r"(smem_u32(tmem_slot)),
                 "r"((uint32_t)kTmemColsF16)
                 : "memory");
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;\n" ::: "memory");
  }
  asm volatile("tcgen05.fence::before_thread_sync;\n" ::: "memory");
  __syncthreads();
  asm volatile("tcgen05.fence::after_thread_sync;\n" ::: "memory");
  const uint32_t tmem_base = *tmem_slot;

  if (warp == 0) {
    if (lane == 0) {   // ---- TMA producer ----
      const uint64_t wpolicy = l2_evict_first_policy();
      int s = 0;
      uint32_t ph = 0;
      for (int kb = 0; kb < nkb; ++kb) {
        if (!mbar_wait(empty + s, ph ^ 1u, abort_flag, a.error)) break;
        unsigned char* st = tiles + s * stage_bytes;
        mbar_expect_tx(full + s, (uint32_t)(kRawBytes + b_bytes));
        tma_load_2d_stream(st + b_bytes, &map_w, k_begin + kb * 64, n0, full + s, wpolicy);                       // 128 rows x 64 int8
        tma_load_2d(st, &map_x, (k_begin + kb * 64) * 2, 0, full + s);                            // Mpad rows x 64 fp16 (byte coordinate)
        if (++s == kStagesF16) { s = 0; ph ^= 1u; }
      }
    }
  } else if (warp == 1) {
    if (lane == 0) {   // ---- MMA issuer ----
      const uint32_t idesc = umma_idesc(/*f32*/ 1, /*fp16*/ 0, a.Mpad);
      int s = 0;
      uint32_t ph = 0;
      bool ok = true;
      for (int kb = 0; kb < nkb && ok; ++kb) {
        if (!(ok = mbar_wait(conv + s, ph, abort_flag, a.error))) break;    // (the converters waited for the stage's TMA)
        asm volatile("tcgen05.fence::after_thread_sync;\n" ::: "memory");
        const uint64_t db = umma_desc_sw128(tiles + s * stage_bytes);
        const uint32_t ta = tmem_base + (uint32_t)(kAccCols + s * kAColsPerStage);
#pragma unroll
        for (int j = 0; j < 4; ++j)   // one instruction contracts 16 fp16 values: 8 columns of A, 32 bytes further along B's rows
          umma_ts_f16(tmem_base, ta + (uint32_t)(j * 8), db + (uint64_t)(j * 2), idesc, (kb > 0 || j > 0) ? 1u : 0u);
        umma_commit(empty + s);
        if (++s == kStagesF16) { s = 0; ph ^= 1u; }
      }
      if (ok) umma_commit(accum_done);
    }
  } else {
    // ---- converters, then the epilogue: warps 2..5; a warp may touch the tensor-memory lanes 32 (warp % 4) .. + 31,
    //      so thread (q, lane) takes weight row r = 32 q + lane of the tile ----
    const int q = warp & 3;
    const int r = q * 32 + lane;
    const uint32_t lane_addr = (uint32_t)(q * 32) << 16;
    int s = 0;
    uint32_t ph = 0;
    bool ok = true;
    for (int kb = 0; kb < nkb; ++kb) {
      int got = 1;
      if (lane == 0) got = mbar_wait(full + s, ph, abort_flag, a.error) ? 1 : 0;
      got = __shfl_sync(0xffffffffu, got, 0);
      if (!got) { ok = false; break; }
      const unsigned char* raw = tiles + s * stage_bytes + b_bytes + r * 64;   // 64-byte swizzle: piece c sits at c ^ ((r >> 1) & 3)
      uint32_t v[32];
#pragma unroll
      for (int c = 0; c < 4; ++c) {
        const uint4 w = *reinterpret_cast<const uint4*>(raw + ((c ^ ((r >> 1) & 3)) << 4));
        s8x4_to_f16x4(w.x, v[8 * c + 0], v[8 * c + 1]);
        s8x4_to_f16x4(w.y, v[8 * c + 2], v[8 * c + 3]);
        s8x4_to_f16x4(w.z, v[8 * c + 4], v[8 * c + 5]);
        s8x4_to_f16x4(w.w, v[8 * c + 6], v[8 * c + 7]);
      }
      tmem_st32(tmem_base + lane_addr + (uint32_t)(kAccCols + s * kAColsPerStage), v);
      asm volatile("tcgen05.fence::before_thread_sync;\n" ::: "memory");
      __syncwarp();
      if (lane == 0) mbar_arrive(conv + s);
      if (++s == kStagesF16) { s = 0; ph ^= 1u; }
    }
    const int n = n0 + r;
    int got = ok ? 1 : 0;
    if (ok && lane == 0) got = mbar_wait(accum_done, 0, abort_flag, a.error) ? 1 : 0;
    got = __shfl_sync(0xffffffffu, got, 0);
    if (got) {
      asm volatile("tcgen05.fence::after_thread_sync;\n" ::: "memory");
      for (int c0 = 0; c0 < a.Mpad; c0 += 16) {
        uint32_t v[16];
        tmem_ld16(tmem_base + lane_addr + (uint32_t)c0, v);
        if (n < a.N) {
#pragma unroll
          for (int j = 0; j < 16; ++j) {
            const int m = c0 + j;
            if (m >= a.M) continue;
            if (a.direct) store_output<false>(a, v[j], m, n);
            else __stcg(reinterpret_cast<uint32_t*>(a.partial) + ((size_t)blockIdx.y * a.Mpad + m) * a.N + n, v[j]);
          }
        }
      }
    }
  }
  asm volatile("tcgen05.fence::before_thread_sync;\n" ::: "memory");
  __threadfence();
  __syncthreads();
  if (warp == 1) {
    asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;\n" ::"r"(tmem_base), "r"((uint32_t)kTmemColsF16)
                 : "memory");
  }
}

// The activation pre-pass of the weight-only form: bf16 row -> fp16 row times a power of two, and the inverse
// of that power for the epilogue.  One CTA per row.
__global__ void __launch_bounds__(256) f16_rows_kernel(const __nv_bfloat16* __restrict__ x, int64_t K, __half* __restrict__ x16,
                                                       float* __restrict__ inv_scale) {
  const int64_t m = blockIdx.x;
  const __nv_bfloat16* row = x + m * K;
  float amax = 0.f;
  for (int64_t k = threadIdx.x; k < K; k += 256) amax = fmaxf(amax, fabsf(__bfloat162float(row[k])));
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) amax = fmaxf(amax, __shfl_xor_sync(0xffffffffu, amax, o));
  __shared__ float s_max[8];
  if ((threadIdx.x & 31) == 0) s_max[threadIdx.x >> 5] = amax;
  __syncthreads();
  amax = s_max[0];
#pragma unroll
  for (int i = 1; i < 8; ++i) amax = fmaxf(amax, s_max[i]);
  float scale, inv;
  f16_row_scale(amax, scale, inv);
  if (threadIdx.x == 0) inv_scale[m] = inv;
  for (int64_t k = threadIdx.x; k < K; k += 256) x16[m * K + k] = __float2half_rn(__bfloat162float(row[k]) * scale);
}

// ---- blocks of at most 8 rows: the weight-only product as an exact integer contraction -------------------
// With so few rows the layer is a pure weight stream, and the cheapest consumer of a weight byte is one that no
// instruction of the SM's own pipelines ever touches: the int8 tile goes from TMA straight into the integer
// MMA (kind::i8).  The 16-bit activations enter as integers too: a row is written as fixed point against a power of
// two above its largest magnitude,  x = q * 2^(E-21)  with |q| <= 2^21, and q as three balanced base-256 digits
// q = d0 + 256 d1 + 65536 d2, each an int8.  A bf16 value has 8 significant bits, so every element within 2^-14 of
// the row's maximum is represented exactly and a smaller one to 2^-22 of that maximum - far inside what an fp32
// accumulation of the same products loses.  The digits are rows of operand B (row 4 m + j = digit j of activation
// row m, j = 3 a zero row), the MMA adds up exact int32 sums per digit (|sum| < 2^31 for up to 2^17 contraction
// bytes per range), and the epilogue puts them together as one 64-bit integer:
//      y[m][n] = delta_w[n] * 2^(E_m - 21) * sum_k w[n][k] q[m][k]        (Section 3.2 Eq. 8 with X kept at 16 bits).
// A CTA is persistent: it keeps the digit rows of one range of the contraction index (<= 2048 bytes: 64 KB)
// resident in shared memory and streams the weight tiles of its share of the channel blocks through an
// eight-stage ring, with two accumulators in tensor memory so that the epilogue of one channel block overlaps the
// MMAs of the next.
constexpr int kStagesS = 8;
constexpr int kDigitKRange = 2048;
constexpr int kStreamTmemCols = 64;

__global__ void __launch_bounds__(256) digit_rows_kernel(const __nv_bfloat16* __restrict__ x, int64_t K, int8_t* __restrict__ xd,
                                                         float* __restrict__ row_scale) {
  const int64_t m = blockIdx.x;
  const __nv_bfloat16* row = x + m * K;
  float amax = 0.f;
  for (int64_t k = threadIdx.x; k < K; k += 256) amax = fmaxf(amax, fabsf(__bfloat162float(row[k])));
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) amax = fmaxf(amax, __shfl_xor_sync(0xffffffffu, amax, o));
  __shared__ float s_max[8];
  if ((threadIdx.x & 31) == 0) s_max[threadIdx.x >> 5] = amax;
  __syncthreads();
  amax = s_max[0];
#pragma unroll
  for (int i = 1; i < 8; ++i) amax = fmaxf(amax, s_max[i]);
  float up = 1.f, down = 1.f;
  if (amax > 0.f && amax < 3.0e38f) {
    int e;
    (void)frexpf(amax, &e);            // amax = f * 2^e, f in [0.5, 1): |x| < 2^e along the row
    e = e < -100 ? -100 : e;           // keeps both factors normal numbers
    up = ldexpf(1.f, 21 - e);
    down = ldexpf(1.f, e - 21);
  } else if (!(amax < 3.0e38f)) {
    down = __int_as_float(0x7fc00000);   // a row holding inf or NaN gives NaN outputs
  }
  if (threadIdx.x == 0) row_scale[m] = down;
  int8_t* d0 = xd + (m * 4 + 0) * K;
  int8_t* d1 = xd + (m * 4 + 1) * K;
  int8_t* d2 = xd + (m * 4 + 2) * K;
  int8_t* d3 = xd + (m * 4 + 3) * K;
  for (int64_t k = threadIdx.x; k < K; k += 256) {
    float v = __bfloat162float(row[k]) * up;
    v = fminf(fmaxf(v, -2097152.f), 2097152.f);
    const int q = __float2int_rn(v);
    const int a0 = (int)(int8_t)(q & 0xff);
    const int q1 = (q - a0) >> 8;
    const int a1 = (int)(int8_t)(q1 & 0xff);
    const int a2 = (q1 - a1) >> 8;
    d0[k] = (int8_t)a0;
    d1[k] = (int8_t)a1;
    d2[k] = (int8_t)a2;
    d3[k] = 0;
  }
}

__global__ void __launch_bounds__(kThreadsU, 1)
umma_stream_kernel(const __grid_constant__ CUtensorMap map_w, const __grid_constant__ CUtensorMap map_xd, UmmaArgs a, int nb,
                   int ctas_per_split, int ntiles) {
  extern __shared__ __align__(16) unsigned char smem_raw[];
  unsigned char* smem = smem_raw + ((1024u - (smem_u32(smem_raw) & 1023u)) & 1023u);
  constexpr int kATile = kTileN * kTileKBytes;
  unsigned char* ring = smem;
  unsigned char* b_res = smem + kStagesS * kATile;                        // digit rows: per 128 contraction bytes nb x 128 B
  uint64_t* full = reinterpret_cast<uint64_t*>(b_res + (size_t)nb * a.k_per_split);
  uint64_t* empty = full + kStagesS;
  uint64_t* b_full = empty + kStagesS;
  uint64_t* acc_full = b_full + 1;     // [2] the MMAs of a channel block have finished
  uint64_t* acc_empty = acc_full + 2;  // [2] the epilogue has read the accumulator out of tensor memory
  uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(acc_empty + 2);
  volatile int* abort_flag = reinterpret_cast<volatile int*>(tmem_slot + 1);

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int split = blockIdx.x / ctas_per_split, part = blockIdx.x % ctas_per_split;
  const int t_begin = (int)((int64_t)part * ntiles / ctas_per_split);
  const int t_end = (int)((int64_t)(part + 1) * ntiles / ctas_per_split);
  const int k_begin = split * a.k_per_split;
  const int k_end = min(a.K, k_begin + a.k_per_split);
  const int nkb = (k_end - k_begin + kTileKBytes - 1) / kTileKBytes;

  if (threadIdx.x == 0) {
    *abort_flag = 0;
    for (int s = 0; s < kStagesS; ++s) {
      mbar_init(full + s, 1);
      mbar_init(empty + s, 1);
    }
    mbar_init(b_full, 1);
    for (int i = 0; i < 2; ++i) {
      mbar_init(acc_full + i, 1);
      mbar_init(acc_empty + i, 4);   // one arrival per epilogue warp
    }
    asm volatile("fence.mbarrier_init.release.cluster;\n" ::: "memory");
  }
  if (warp == 1) {
    asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;\n" ::"r"(smem_u32(tmem_slot)),
                 "r"((uint32_t)kStreamTmemCols)
                 : "memory");
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;\n" ::: "memory");
  }
  asm volatile("tcgen05.fence::before_thread_sync;\n" ::: "memory");
  __syncthreads();
  asm volatile("tcgen05.fence::after_thread_sync;\n" ::: "memory");
  const uint32_t tmem_base = *tmem_slot;

  if (warp == 0) {
    if (lane == 0) {   // ---- TMA producer: the digit rows once, then the weight tiles of every channel block ----
      const uint64_t wpolicy = l2_evict_first_policy();
      mbar_expect_tx(b_full, (uint32_t)(nkb * nb * kTileKBytes));
      for (int kb = 0; kb < nkb; ++kb)
        tma_load_2d(b_res + (size_t)kb * nb * kTileKBytes, &map_xd, k_begin + kb * kTileKBytes, 0, b_full);
      int s = 0;
      uint32_t ph = 0;
      bool ok = true;
      for (int t = t_begin; t < t_end && ok; ++t) {
        for (int kb = 0; kb < nkb; ++kb) {
          if (!(ok = mbar_wait(empty + s, ph ^ 1u, abort_flag, a.error))) break;
          mbar_expect_tx(full + s, (uint32_t)kATile);
          tma_load_2d_stream(ring + s * kATile, &map_w, k_begin + kb * kTileKBytes, t * kTileN, full + s, wpolicy);
          if (++s == kStagesS) { s = 0; ph ^= 1u; }
        }
      }
    }
  } else if (warp == 1) {
    if (lane == 0) {   // ---- MMA issuer ----
      const uint32_t idesc = umma_idesc(/*s32*/ 2, /*signed int8*/ 1, nb);
      int s = 0;
      uint32_t ph = 0;
      bool ok = mbar_wait(b_full, 0, abort_flag, a.error);
      for (int t = t_begin, it = 0; t < t_end && ok; ++t, ++it) {
        const int buf = it & 1;
        if (!(ok = mbar_wait(acc_empty + buf, (((uint32_t)it >> 1) & 1u) ^ 1u, abort_flag, a.error))) break;
        asm volatile("tcgen05.fence::after_thread_sync;\n" ::: "memory");
        const uint32_t tmem_d = tmem_base + (uint32_t)(buf * 32);
        for (int kb = 0; kb < nkb; ++kb) {
          if (!(ok = mbar_wait(full + s, ph, abort_flag, a.error))) break;
          asm volatile("tcgen05.fence::after_thread_sync;\n" ::: "memory");
          const uint64_t da = umma_desc_sw128(ring + s * kATile);
          const uint64_t db = umma_desc_sw128(b_res + (size_t)kb * nb * kTileKBytes);
#pragma unroll
          for (int j = 0; j < kTileKBytes / 32; ++j)
            umma_ss<true>(tmem_d, da + (uint64_t)(j * 2), db + (uint64_t)(j * 2), idesc, (kb > 0 || j > 0) ? 1u : 0u);
          umma_commit(empty + s);
          if (++s == kStagesS) { s = 0; ph ^= 1u; }
        }
        if (ok) umma_commit(acc_full + buf);
      }
    }
  } else {
    // ---- epilogue: warps 2..5, one output channel per thread ----
    const int q = warp & 3;
    for (int t = t_begin, it = 0; t < t_end; ++t, ++it) {
      const int buf = it & 1;
      int got = 1;
      if (lane == 0) got = mbar_wait(acc_full + buf, ((uint32_t)it >> 1) & 1u, abort_flag, a.error) ? 1 : 0;
      got = __shfl_sync(0xffffffffu, got, 0);
      if (!got) break;
      asm volatile("tcgen05.fence::after_thread_sync;\n" ::: "memory");
      uint32_t v0[16], v1[16];
      const uint32_t taddr = tmem_base + ((uint32_t)(q * 32) << 16) + (uint32_t)(buf * 32);
      tmem_ld16(taddr, v0);
      if (nb > 16) tmem_ld16(taddr + 16u, v1);
      asm volatile("tcgen05.fence::before_thread_sync;\n" ::: "memory");
      __syncwarp();
      if (lane == 0) mbar_arrive(acc_empty + buf);     // the next channel block but one may overwrite the accumulator
      const int n = t * kTileN + q * 32 + lane;
      if (n < a.N) {
#pragma unroll
        for (int m = 0; m < 8; ++m) {
          if (m >= a.M) continue;
          const uint32_t* v = m < 4 ? v0 + 4 * m : v1 + 4 * (m - 4);
          const long long total = ((long long)(int)v[2] << 16) + ((long long)(int)v[1] << 8) + (long long)(int)v[0];
          const uint32_t bits = __float_as_uint((float)total);
          if (a.direct) store_output<false>(a, bits, m, n);
          else __stcg(reinterpret_cast<uint32_t*>(a.partial) + ((size_t)split * a.Mpad + m) * a.N + n, bits);
        }
      }
    }
  }
  asm volatile("tcgen05.fence::before_thread_sync;\n" ::: "memory");
  __threadfence();
  __syncthreads();
  if (warp == 1) {
    asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;\n" ::"r"(tmem_base), "r"((uint32_t)kStreamTmemCols)
                 : "memory");
  }
}

// ---- host side ------------------------------------------------------------------------------------
PFN_cuTensorMapEncodeTiled_v12000 encode_fn() {
  static PFN_cuTensorMapEncodeTiled_v12000 fn = nullptr;
  static std::once_flag once;
  std::call_once(once, [] {
    void* p = nullptr;
    cudaDriverEntryPointQueryResult qres;
    if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &p, cudaEnableDefault, &qres) == cudaSuccess &&
        qres == cudaDriverEntryPointSuccess)
      fn = reinterpret_cast<PFN_cuTensorMapEncodeTiled_v12000>(p);
  });
  return fn;
}

// [rows][row_bytes] bytes, box = box_rows x box_bytes (128 with the 128-byte swizzle, 64 with the 64-byte one),
// zeros outside
int make_map(CUtensorMap* map, const void* base, uint64_t rows, uint64_t row_bytes, uint32_t box_rows,
             uint32_t box_bytes = kTileKBytes) {
  auto fn = encode_fn();
  if (fn == nullptr) {
    set_error("cuTensorMapEncodeTiled is not available from this driver");
    return QUASAR_ERR_CUDA;
  }
  const cuuint64_t dims[2] = {row_bytes, rows};
  const cuuint64_t strides[1] = {row_bytes};
  const cuuint32_t box[2] = {(cuuint32_t)box_bytes, box_rows};
  const cuuint32_t estr[2] = {1, 1};
  const CUresult r = fn(map, CU_TENSOR_MAP_DATA_TYPE_UINT8, 2, const_cast<void*>(base), dims, strides, box, estr,
                        CU_TENSOR_MAP_INTERLEAVE_NONE, box_bytes == 64 ? CU_TENSOR_MAP_SWIZZLE_64B : CU_TENSOR_MAP_SWIZZLE_128B,
                        CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                        CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
  if (r != CUDA_SUCCESS) {
    set_error("cuTensorMapEncodeTiled failed (%d) for %llu x %llu bytes", (int)r, (unsigned long long)rows,
              (unsigned long long)row_bytes);
    return QUASAR_ERR_CUDA;
  }
  return QUASAR_OK;
}

struct SplitU {
  int nblocks, nsplit, k_per_split;
};
SplitU plan_split_u(int64_t N, int64_t K) {
  SplitU p;
  p.nblocks = (int)((N + kTileN - 1) / kTileN);
  const int kbs = (int)((K + kTileKBytes - 1) / kTileKBytes);
  int want = 296 / p.nblocks;                          // about two CTAs per SM (what its shared memory holds); no split once the channel blocks fill them
  want = want < 1 ? 1 : (want > kbs ? kbs : want);
  want = want > 32 ? 32 : want;
  const int per = (kbs + want - 1) / want;
  p.k_per_split = per * kTileKBytes;
  p.nsplit = (kbs + per - 1) / per;
  return p;
}

}  // namespace

bool umma_w8a8_usable(int64_t M, int64_t N, int64_t K) {
  return M > 8 && M <= kMaxMpad && K % 16 == 0 && N >= 1 && (int64_t)((N + kTileN - 1) / kTileN) * 4 <= (int64_t)kCounterBytesU;
}

size_t umma_w8a8_partial_bytes(int64_t M, int64_t N, int64_t K) {
  const SplitU p = plan_split_u(N, K);
  const size_t mpad = (size_t)((M + 15) / 16) * 16;
  return p.nsplit > 1 ? (size_t)p.nsplit * mpad * (size_t)N * 4 : 0;
}

// xq: int8 [M][K] quantised activations, dx their step sizes; counters: >= 64 KiB, zero on first use
int launch_umma_w8a8(const int8_t* xq, const float* dx, const int8_t* w, const float* dw, int64_t M, int64_t N, int64_t K,
                     void* y, bool y_is_f32, const __nv_bfloat16* residual, int32_t* acc_out, int* counters, void* partial,
                     int32_t* error_word, cudaStream_t stream) {
  CUtensorMap map_w, map_x;
  const int mpad = (int)((M + 15) / 16) * 16;
  int rc = make_map(&map_w, w, (uint64_t)N, (uint64_t)K, kTileN);
  if (rc != QUASAR_OK) return rc;
  rc = make_map(&map_x, xq, (uint64_t)M, (uint64_t)K, (uint32_t)mpad);
  if (rc != QUASAR_OK) return rc;
  const SplitU p = plan_split_u(N, K);
  UmmaArgs a;
  a.dx = dx; a.dw = dw; a.y = y; a.res = residual; a.acc_out = acc_out; a.partial = partial; a.counters = counters;
  a.error = error_word;
  a.M = (int)M; a.Mpad = mpad; a.N = (int)N; a.K = (int)K; a.k_per_split = p.k_per_split; a.nsplit = p.nsplit;
  a.y_is_f32 = y_is_f32 ? 1 : 0;
  a.direct = p.nsplit == 1 ? 1 : 0;
  const size_t smem = (size_t)kStagesI8 * (kTileN * kTileKBytes + mpad * kTileKBytes) + 256 + 1024;
  static bool configured = false;
  if (!configured) {
    QUASAR_CUDA_CHECK(cudaFuncSetAttribute(umma_gemm_kernel<true>, cudaFuncAttributeMaxDynamicSharedMemorySize, 112 * 1024));
    configured = true;
  }
  umma_gemm_kernel<true><<<dim3(p.nblocks, p.nsplit), kThreadsU, smem, stream>>>(map_w, map_x, a);
  QUASAR_LAUNCH_CHECK();
  if (p.nsplit > 1) {
    const int64_t items = M * ((N + 3) / 4);
    umma_reduce_kernel<true><<<(unsigned)((items + 255) / 256), 256, 0, stream>>>(a);
    QUASAR_LAUNCH_CHECK();
  }
  return QUASAR_OK;
}


// ---- weight-only form ----
bool umma_w8a16_usable(int64_t M, int64_t N, int64_t K) {
  return M > 8 && M <= kMaxMpad && K % 16 == 0 && N >= 1;
}

void umma_w8a16_plan(int64_t M, int64_t N, int64_t K, int* nsplit, int* mpad) {
  *nsplit = plan_split_u(N, K).nsplit;
  *mpad = (int)((M + 15) / 16) * 16;
}

// bytes of the partial sums (also when one k-range is asked to leave its sums for a fused consumer, unless the
// matrix is as wide as an LM head, which always finishes itself)
size_t umma_w8a16_partial_bytes(int64_t M, int64_t N, int64_t K) {
  const SplitU p = plan_split_u(N, K);
  const size_t mpad = (size_t)((M + 15) / 16) * 16;
  return (p.nsplit > 1 || N <= 32768) ? (size_t)p.nsplit * mpad * (size_t)N * 4 : 0;
}

// bytes of scratch: fp16 copy of the activation rows, their inverse scales, partial sums of the k-ranges
size_t umma_w8a16_scratch_bytes(int64_t M, int64_t N, int64_t K) {
  return ((size_t)M * K * 2 + 255) / 256 * 256 + ((size_t)M * 4 + 255) / 256 * 256 + umma_w8a16_partial_bytes(M, N, K);
}

int launch_f16_rows(const __nv_bfloat16* x, int64_t M, int64_t K, void* x16, float* inv_scale, cudaStream_t stream) {
  f16_rows_kernel<<<(unsigned)M, 256, 0, stream>>>(x, K, reinterpret_cast<__half*>(x16), inv_scale);
  QUASAR_LAUNCH_CHECK();
  return QUASAR_OK;
}

// x16 / inv: the activation rows as fp16 times a power of two and the inverse of that power (f16_rows_kernel or a
// producer that writes the same thing).  finalize = false leaves the partial sums of every k-range in `partial`
// ([nsplit][mpad][N] fp32, see umma_w8a16_plan) for a consumer that adds them up itself.
int launch_umma_w8a16_prepared(const void* x16, const float* inv, const int8_t* w, const float* dw, int64_t M, int64_t N,
                               int64_t K, void* y, bool y_is_f32, const __nv_bfloat16* residual, void* partial, bool finalize,
                               int32_t* error_word, cudaStream_t stream) {
  CUtensorMap map_w, map_x;
  const int mpad = (int)((M + 15) / 16) * 16;
  int rc = make_map(&map_w, w, (uint64_t)N, (uint64_t)K, kTileN, 64);
  if (rc != QUASAR_OK) return rc;
  rc = make_map(&map_x, x16, (uint64_t)M, (uint64_t)K * 2, (uint32_t)mpad, 128);
  if (rc != QUASAR_OK) return rc;
  const SplitU p = plan_split_u(N, K);
  UmmaArgs a;
  a.dx = inv; a.dw = dw; a.y = y; a.res = residual; a.acc_out = nullptr; a.partial = partial; a.counters = nullptr;
  a.error = error_word;
  a.M = (int)M; a.Mpad = mpad; a.N = (int)N; a.K = (int)K; a.k_per_split = p.k_per_split; a.nsplit = p.nsplit;
  a.y_is_f32 = y_is_f32 ? 1 : 0;
  a.direct = (finalize && p.nsplit == 1) ? 1 : 0;
  const size_t smem = (size_t)kStagesF16 * (mpad * 128 + kRawBytes) + 256 + 1024;
  static bool configured = false;
  if (!configured) {
    QUASAR_CUDA_CHECK(cudaFuncSetAttribute(umma_w8a16_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, 112 * 1024));
    configured = true;
  }
  umma_w8a16_kernel<<<dim3(p.nblocks, p.nsplit), kThreadsU, smem, stream>>>(map_w, map_x, a);
  QUASAR_LAUNCH_CHECK();
  if (finalize && p.nsplit > 1) {
    const int64_t items = M * ((N + 3) / 4);
    umma_reduce_kernel<false><<<(unsigned)((items + 255) / 256), 256, 0, stream>>>(a);
    QUASAR_LAUNCH_CHECK();
  }
  return QUASAR_OK;
}

int launch_umma_w8a16(const __nv_bfloat16* x, const int8_t* w, const float* dw, int64_t M, int64_t N, int64_t K, void* y,
                      bool y_is_f32, const __nv_bfloat16* residual, void* scratch, int32_t* error_word, cudaStream_t stream) {
  unsigned char* sc = reinterpret_cast<unsigned char*>(scratch);
  float* inv = reinterpret_cast<float*>(sc + ((size_t)M * K * 2 + 255) / 256 * 256);
  void* partial = sc + ((size_t)M * K * 2 + 255) / 256 * 256 + ((size_t)M * 4 + 255) / 256 * 256;
  int rc = launch_f16_rows(x, M, K, sc, inv, stream);
  if (rc != QUASAR_OK) return rc;
  return launch_umma_w8a16_prepared(sc, inv, w, dw, M, N, K, y, y_is_f32, residual, partial, true, error_word, stream);
}

// ---- weight-only form, at most 8 rows ----
namespace {
struct StreamPlan {
  int nb, nsplit, k_per_split, ntiles, ctas_per_split;
};
StreamPlan plan_stream(int64_t M, int64_t N, int64_t K) {
  StreamPlan p;
  p.nb = M <= 4 ? 16 : 32;
  const int kbs = (int)((K + kTileKBytes - 1) / kTileKBytes);
  const int want = (int)((K + kDigitKRange - 1) / kDigitKRange);
  const int per = (kbs + want - 1) / want;
  p.k_per_split = per * kTileKBytes;
  p.nsplit = (kbs + per - 1) / per;
  p.ntiles = (int)((N + kTileN - 1) / kTileN);
  int cps = 148 / p.nsplit;
  cps = cps < 1 ? 1 : cps;
  p.ctas_per_split = cps < p.ntiles ? cps : p.ntiles;
  return p;
}
}  // namespace

bool umma_rows8_usable(int64_t M, int64_t N, int64_t K) {
  return M >= 1 && M <= 8 && K % 16 == 0 && N >= 1 && K <= (int64_t)148 * kDigitKRange;
}

// bytes of scratch: the digit rows, the rows' scales, partial sums of the k-ranges
size_t umma_rows8_scratch_bytes(int64_t M, int64_t N, int64_t K) {
  const StreamPlan p = plan_stream(M, N, K);
  const size_t partial = p.nsplit > 1 ? (size_t)p.nsplit * (size_t)M * (size_t)N * 4 : 0;
  return ((size_t)4 * M * K + 255) / 256 * 256 + 256 + partial;
}

int launch_umma_rows8(const __nv_bfloat16* x, const int8_t* w, const float* dw, int64_t M, int64_t N, int64_t K, void* y,
                      bool y_is_f32, const __nv_bfloat16* residual, void* scratch, int32_t* error_word, cudaStream_t stream) {
  unsigned char* sc = reinterpret_cast<unsigned char*>(scratch);
  int8_t* xd = reinterpret_cast<int8_t*>(sc);
  float* row_scale = reinterpret_cast<float*>(sc + ((size_t)4 * M * K + 255) / 256 * 256);
  void* partial = sc + ((size_t)4 * M * K + 255) / 256 * 256 + 256;
  digit_rows_kernel<<<(unsigned)M, 256, 0, stream>>>(x, K, xd, row_scale);
  QUASAR_LAUNCH_CHECK();
  const StreamPlan p = plan_stream(M, N, K);
  CUtensorMap map_w, map_xd;
  int rc = make_map(&map_w, w, (uint64_t)N, (uint64_t)K, kTileN);
  if (rc != QUASAR_OK) return rc;
  rc = make_map(&map_xd, xd, (uint64_t)(4 * M), (uint64_t)K, (uint32_t)p.nb);
  if (rc != QUASAR_OK) return rc;
  UmmaArgs a;
  a.dx = row_scale; a.dw = dw; a.y = y; a.res = residual; a.acc_out = nullptr; a.partial = partial; a.counters = nullptr;
  a.error = error_word;
  a.M = (int)M; a.Mpad = (int)M; a.N = (int)N; a.K = (int)K; a.k_per_split = p.k_per_split; a.nsplit = p.nsplit;
  a.y_is_f32 = y_is_f32 ? 1 : 0;
  a.direct = p.nsplit == 1 ? 1 : 0;
  const size_t smem = (size_t)kStagesS * kTileN * kTileKBytes + (size_t)p.nb * p.k_per_split + 256 + 1024;
  static bool configured = false;
  if (!configured) {
    QUASAR_CUDA_CHECK(cudaFuncSetAttribute(umma_stream_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, 200 * 1024));
    configured = true;
  }
  umma_stream_kernel<<<(unsigned)(p.nsplit * p.ctas_per_split), kThreadsU, smem, stream>>>(map_w, map_xd, a, p.nb,
                                                                                         p.ctas_per_split, p.ntiles);
  QUASAR_LAUNCH_CHECK();
  if (p.nsplit > 1) {
    const int64_t items = M * ((N + 3) / 4);
    umma_reduce_kernel<false><<<(unsigned)((items + 255) / 256), 256, 0, stream>>>(a);
    QUASAR_LAUNCH_CHECK();
  }
  return QUASAR_OK;
}

}  // namespace quasar
