// The whole verification pass (Section 3.1 "Verification", Section 3.3) as ONE persistent
// cooperative kernel: one CTA per SM, every step of the pass a phase separated by a grid
// barrier.  Section 3.4 models the pass as  T ~= M * bytes / BW : the pass is one long read
// of the weights, so the design goal is that this read never stops.
//
//  * Each weight matrix is cut into contiguous row ranges, one per CTA, balanced to a single
//    row, so all SMs stream the same number of bytes and no cross-CTA reduction exists.
//    Inside a CTA the 8 consumer warps split the contraction index; their partial sums meet
//    in shared memory in a fixed order (deterministic results).
//  * At model creation the bytes of every CTA's row range are permuted (same size, same
//    place) into the order in which that CTA consumes them: blocks of <= 16 rows x 1024
//    bytes, each block contiguous, 16-byte pieces XOR-swizzled for conflict-free 128-bit
//    shared-memory reads, int8 sign bits pre-flipped.  A ring stage is then ONE bulk
//    asynchronous copy (cp.async.bulk) of up to 16 KB from a pointer that only moves forward:
//    measured on B200, 16 KB copies stream at 6.2-7.0 TB/s where 1 KB row pieces reach 2.9 TB/s
//    (the copy engine's cost is per request).
//  * A dedicated producer warp walks a STATIC schedule covering every GEMM of the pass and
//    fills the ring (completion counted in bytes by an mbarrier per stage).  The schedule
//    does not depend on activations, so the producer keeps prefetching the next GEMM's
//    weights while the consumer warps are in an epilogue, an attention phase or a grid
//    barrier (128 KB in flight per SM), and loading costs the consumers no instructions.
//  * int8 -> fp16 in registers at one instruction per two weights: the byte, stored with its sign
//    bit flipped, becomes the low mantissa byte of the fp16 number 1024 + (w + 128), and one
//    packed subtraction of 1152 leaves w exactly.  The activations are bf16 values converted
//    to fp16 (exact; a per-row power-of-two pre-scale keeps any bf16 row inside the fp16
//    range), so mma.m16n8k16 f16 x f16 -> f32 computes the same products the bf16 operands
//    would.  The weights are the 16-row operand, the <= 8 activation rows the 8-wide operand:
//    they are brought into shared memory by bulk copy at the head of a phase, converted there
//    once, and every stage reads its slice of them (the stage loop is rolled so that its code
//    stays in the instruction cache).  The o and down projections find their operands already
//    as fp16, written beside the bf16 tensors by the phases that produce them.
//  * RMSNorm is fused into the operand load of the following GEMM, SwiGLU / residual adds
//    into the GEMM epilogues, QK-RMSNorm + RoPE + KV append into the attention phase.
//
// Every wait is bounded: a grid barrier or an mbarrier that does not complete within its
// time budget sets QUASAR_ERR_TIMEOUT in the status word and the CTA leaves (after its own
// copies in flight have landed).
#include <cooperative_groups.h>
#include <math.h>

#include "common.cuh"
#include "megakernel.cuh"

namespace quasar {

namespace {

constexpr int NW = kMegaWarps;             // consumer warps per CTA
constexpr int kCT = NW * 32;               // consumer threads
constexpr int kThreads = kCT + 32;         // + the producer warp (9 warps: at most 3 per SM sub-partition, so 168 registers per thread)
constexpr int kRowBytes = 1024;            // bytes of one weight row per stage
constexpr int kStageBytes = 16 * kRowBytes;  // 16 weight rows
constexpr int kStages = 8;                 // ring depth (128 KB of weights in flight per CTA)
constexpr int kChunk = 4096;               // longest contraction whose operand rows stay in shared memory whole
constexpr int kChunkLong = 2048;           // chunk of a longer contraction: two operand buffers, one in use while the next lands
constexpr int kWarpBytes = kRowBytes / NW;   // bytes of a row piece one warp covers (128)
constexpr int kSub = kWarpBytes / 64;        // 64-byte sub-slices of it: four lanes x 16 bytes each
constexpr int GT = 4;                      // 16-row tiles accumulated together before a reduction
constexpr int kKeyTile = 64;
constexpr int kMaxRowsAttn = 32;           // query rows (heads-in-group x block rows) per kv head
constexpr float kLog2e = 1.4426950408889634f;

// ---- shared memory map --------------------------------------------------------------------
constexpr int kRingBytes = kStages * kStageBytes;                        // 131072
constexpr int kRedBytes = NW * GT * 128 * 4;                             // 16384
constexpr int kKvTileBytes = kKeyTile * (128 + 8) * 2;                   // 17408 (D = 128)
constexpr int kQTileBytes = kMaxRowsAttn * (128 + 8) * 2;                // 17408
constexpr int kOTileBytes = kMaxRowsAttn * 128 * 4;                      // 16384: a CTA's partial output before it is stored
constexpr int kMlTileBytes = kMaxRowsAttn * 8;                           // its row maxima and sums
constexpr int kAttnBytes = 2 * kKvTileBytes + kQTileBytes + kOTileBytes + kMlTileBytes;   // tiles of the attention phase
constexpr int kMiscBytes = 2048;
// The operand of a GEMM phase (<= 8 rows x one chunk) and its norm gain land in a staging buffer by bulk
// copy, are converted there and stay there while the phase multiplies: every stage reads its slice of
// the rows from it.  Rows sit at a pitch of the chunk's bytes plus a pad that spreads the rows over the
// banks.  A contraction longer than kChunk goes through two half-size buffers in turn.  The attention
// tiles share the bytes: the two are never alive at the same time.  The reduction buffer has bytes of
// its own.
constexpr int kXPadInt8 = 16, kXPadBf16 = 64;
constexpr int kXBufWhole = 8 * (kChunk * 2 + kXPadBf16) + kChunk * 2;            // rows + gain: 74240
constexpr int kXBufLong = 8 * (kChunkLong * 2 + kXPadBf16) + kChunkLong * 2;     // 37376, twice
constexpr int kXBufBytes = kXBufWhole > 2 * kXBufLong ? kXBufWhole : 2 * kXBufLong;
constexpr int kStageBufBytes = kXBufBytes > kAttnBytes ? kXBufBytes : kAttnBytes;
constexpr int kSmemBytes = kRingBytes + kRedBytes + kStageBufBytes + kMiscBytes;
static_assert(kSmemBytes <= 227 * 1024, "shared memory budget of one SM");

// misc region (floats): [0,128) per-warp row sums, [128,136) running arg-max values, [136,144) its
// indices, [144,152) 1/scale of the operand rows, [152,184) per-tile sums of squares, [200] abort flag, [256,512) candidates / per-warp
// row maxima, byte 1536.. the mbarriers.
constexpr int kMiscRowSum = 0, kMiscRunV = 128, kMiscRunI = 136, kMiscInvScale = 144, kMiscPart = 152, kMiscFlag = 190, kMiscRs = 192, kMiscAbort = 200, kMiscJob = 208 /* two descriptors of 40 bytes */,
              kMiscCand = 256, kMiscBarBytes = 1536;   // 2 kStages + 1 barriers of 8 bytes

__device__ __forceinline__ void mma16816_bf16(float (&c)[4], uint32_t a0, uint32_t a1, uint32_t a2, uint32_t a3,
                                              uint32_t b0, uint32_t b1) {
  asm volatile(
      "mma.sync.aligned.m16n8k16.row.col.f32.bf16.bf16.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%0,%1,%2,%3};\n"
      : "+f"(c[0]), "+f"(c[1]), "+f"(c[2]), "+f"(c[3])
      : "r"(a0), "r"(a1), "r"(a2), "r"(a3), "r"(b0), "r"(b1));
}
__device__ __forceinline__ void mma16816_f16(float (&c)[4], uint32_t a0, uint32_t a1, uint32_t a2, uint32_t a3,
                                             uint32_t b0, uint32_t b1) {
  asm volatile(
      "mma.sync.aligned.m16n8k16.row.col.f32.f16.f16.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%0,%1,%2,%3};\n"
      : "+f"(c[0]), "+f"(c[1]), "+f"(c[2]), "+f"(c[3])
      : "r"(a0), "r"(a1), "r"(a2), "r"(a3), "r"(b0), "r"(b1));
}

__device__ __forceinline__ void ldmatrix_x4_trans(uint32_t& r0, uint32_t& r1, uint32_t& r2, uint32_t& r3,
                                                  const void* smem_ptr) {
  const uint32_t addr = (uint32_t)__cvta_generic_to_shared(smem_ptr);
  asm volatile("ldmatrix.sync.aligned.m8n8.x4.trans.shared.b16 {%0,%1,%2,%3}, [%4];\n"
               : "=r"(r0), "=r"(r1), "=r"(r2), "=r"(r3)
               : "r"(addr));
}

// Four weight bytes -> four fp16 (exact).  The repacked bytes hold u = w + 128 in [1, 255]
// (sign bit flipped); placed under the high byte 0x64, u reads 1024 + u as fp16 (the spacing of
// fp16 in [1024, 2048) is 1), and subtracting 1152 leaves w.  lo = bytes 0,1; hi = bytes 2,3.
__device__ __forceinline__ void u8x4_to_f16x4(uint32_t u, uint32_t& lo, uint32_t& hi) {
  const uint32_t l = __byte_perm(u, 0x64646464u, 0x4140);
  const uint32_t h = __byte_perm(u, 0x64646464u, 0x4342);
  const __half2 bias = __halves2half2(__ushort_as_half(0x6480), __ushort_as_half(0x6480));
  const __half2 lo2 = __hsub2(*reinterpret_cast<const __half2*>(&l), bias);
  const __half2 hi2 = __hsub2(*reinterpret_cast<const __half2*>(&h), bias);
  lo = *reinterpret_cast<const uint32_t*>(&lo2);
  hi = *reinterpret_cast<const uint32_t*>(&hi2);
}

__device__ __forceinline__ uint32_t pack_bf16(float lo, float hi) {
  __nv_bfloat162 p = __floats2bfloat162_rn(lo, hi);
  return *reinterpret_cast<uint32_t*>(&p);
}
__device__ __forceinline__ void split_bf16(float a, float b, uint32_t& hi, uint32_t& lo) {
  const __nv_bfloat16 ah = __float2bfloat16_rn(a), bh = __float2bfloat16_rn(b);
  __nv_bfloat162 h;
  h.x = ah;
  h.y = bh;
  hi = *reinterpret_cast<uint32_t*>(&h);
  lo = pack_bf16(a - __bfloat162float(ah), b - __bfloat162float(bh));
}
__device__ __forceinline__ float bf16_round_f(float v) { return __bfloat162float(__float2bfloat16_rn(v)); }
__device__ __forceinline__ float warp_sum(float v) {
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
  return v;
}

// Loads that must be ISSUED where they are written (the compiler may not sink them to their first use):
// the epilogue's step sizes and residual are requested before the stage loop and arrive during it.
__device__ __forceinline__ float ld_early_f32(const float* p) {
  float v;
  asm volatile("ld.global.nc.f32 %0, [%1];\n" : "=f"(v) : "l"(p));
  return v;
}
__device__ __forceinline__ float ld_early_bf16_cg(const __nv_bfloat16* p) {
  unsigned short v;
  asm volatile("ld.global.cg.u16 %0, [%1];\n" : "=h"(v) : "l"(p));
  return __uint_as_float((unsigned)v << 16);
}

// barrier among the consumer warps only (the producer warp never joins it)
__device__ __forceinline__ void cbar() { asm volatile("bar.sync 1, %0;\n" ::"n"(kCT) : "memory"); }

__device__ __forceinline__ unsigned long long now_ns() {
  unsigned long long t;
  asm volatile("mov.u64 %0, %%globaltimer;\n" : "=l"(t));
  return t;
}


// ---- mbarriers ----------------------------------------------------------------------------
__device__ __forceinline__ void mbar_init(uint64_t* bar, int count) {
  asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;\n" ::"r"((uint32_t)__cvta_generic_to_shared(bar)), "r"(count)
               : "memory");
}
__device__ __forceinline__ void mbar_arrive(uint64_t* bar) {
  asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];\n" ::"r"((uint32_t)__cvta_generic_to_shared(bar)) : "memory");
}
__device__ __forceinline__ void mbar_arrive_expect_tx(uint64_t* bar, uint32_t bytes) {
  asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;\n" ::"r"((uint32_t)__cvta_generic_to_shared(bar)),
               "r"(bytes)
               : "memory");
}
__device__ __forceinline__ bool mbar_try(uint64_t* bar, uint32_t parity) {
  uint32_t ok;
  asm volatile(
      "{\n.reg .pred p;\nmbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\nselp.u32 %0, 1, 0, p;\n}\n"
      : "=r"(ok)
      : "r"((uint32_t)__cvta_generic_to_shared(bar)), "r"(parity)
      : "memory");
  return ok != 0;
}
// Waits for the phase of `bar` with the given parity.  Gives up when another thread of the CTA
// has raised the abort flag or after the launch's wait budget (then raises the flag and the status itself).
// The budget sits in shared memory two words behind the abort flag.
__device__ __forceinline__ unsigned long long wait_budget(volatile int* abort_flag) {
  return *reinterpret_cast<volatile unsigned long long*>(abort_flag + 2);
}
__device__ __noinline__ bool mbar_wait_slow(uint64_t* bar, uint32_t parity, volatile int* abort_flag, int32_t* status) {
  const unsigned long long t0 = now_ns();
  unsigned it = 0;
  while (true) {
    if (mbar_try(bar, parity)) return true;
    if ((++it & 63u) == 0) {
      if (*abort_flag) return false;
      if (now_ns() - t0 > wait_budget(abort_flag)) {
        atomicMin(status, QUASAR_ERR_TIMEOUT);
        *abort_flag = 1;
        return false;
      }
    }
  }
}
__device__ __forceinline__ bool mbar_wait(uint64_t* bar, uint32_t parity, volatile int* abort_flag, int32_t* status) {
  if (mbar_try(bar, parity)) return true;
  return mbar_wait_slow(bar, parity, abort_flag, status);
}

// One block of weights (a multiple of 16 bytes, both addresses 16-byte aligned) from global to
// shared memory; completion is counted in bytes on `bar`.  The weights are read once per pass, so
// the copy asks L2 to evict them first.
__device__ __forceinline__ void bulk_copy(void* smem_dst, const void* gmem_src, uint32_t bytes, uint64_t* bar,
                                              uint64_t policy) {
  asm volatile(
      "cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes.L2::cache_hint [%0], [%1], %2, [%3], %4;\n" ::"r"(
          (uint32_t)__cvta_generic_to_shared(smem_dst)),
      "l"(gmem_src), "r"(bytes), "r"((uint32_t)__cvta_generic_to_shared(bar)), "l"(policy)
      : "memory");
}

// ---- the static weight schedule -----------------------------------------------------------
// Order of the ring stages of the whole pass, identical for the producer, the consumers and
// the repacked weight layout:  job -> tile group -> contraction chunk -> tile in group ->
// 1024-byte piece of the chunk.  A stage holds one block: the rows of one tile (<= 16) x one
// piece, rows at a pitch of the piece's bytes.
struct JobView {
  const unsigned char* wp;   // this CTA's repacked row range
  int K, units, u0, u1, rows_per_tile, tiles, ngroups, nchunks, chunk, kind, n_rows;
};

__device__ __forceinline__ void job_split(int kind, int N, int K, int cta, int ncta, JobView& v) {
  v.K = K;
  v.kind = kind;
  v.n_rows = N;
  v.units = (kind == kJobGateUp) ? N / 2 : N;
  v.u0 = (int)(((long long)cta * v.units) / ncta);
  v.u1 = (int)(((long long)(cta + 1) * v.units) / ncta);
  v.rows_per_tile = (kind == kJobGateUp) ? 8 : 16;
  v.tiles = (v.u1 - v.u0 + v.rows_per_tile - 1) / v.rows_per_tile;
  v.ngroups = (v.tiles + GT - 1) / GT;
  v.chunk = K <= kChunk ? K : kChunkLong;   // contraction elements per chunk
  v.nchunks = (K + v.chunk - 1) / v.chunk;
}

template <bool W_INT8>
__device__ __forceinline__ JobView job_view_of(const MegaJob& jb, int cta, int ncta) {
  JobView v;
  job_split(jb.kind, jb.N, jb.K, cta, ncta, v);
  const size_t row_bytes = (size_t)jb.K * (W_INT8 ? 1 : 2);
  v.wp = reinterpret_cast<const unsigned char*>(jb.wp) + (size_t)(jb.kind == kJobGateUp ? 2 * v.u0 : v.u0) * row_bytes;
  return v;
}
template <bool W_INT8>
__device__ __forceinline__ JobView job_view(const MegaJob* jobs, int j, int cta, int ncta) {
  JobView v;
  const MegaJob jb = jobs[j];
  job_split(jb.kind, jb.N, jb.K, cta, ncta, v);
  const size_t row_bytes = (size_t)jb.K * (W_INT8 ? 1 : 2);
  v.wp = reinterpret_cast<const unsigned char*>(jb.wp) + (size_t)(jb.kind == kJobGateUp ? 2 * v.u0 : v.u0) * row_bytes;
  return v;
}

// units (output channels, or gate/up pairs) of tile `tile` of this CTA, and rows of its blocks
__device__ __forceinline__ int tile_units(const JobView& v, int tile) {
  return min(v.rows_per_tile, v.u1 - v.u0 - tile * v.rows_per_tile);
}
__device__ __forceinline__ int tile_rows(const JobView& v, int tile) {
  const int u = tile_units(v, tile);
  return v.kind == kJobGateUp ? 2 * u : u;
}
// global weight row stored in row `r` of the blocks of tile `tile` (r < tile_rows): a gate/up
// tile keeps its gate rows first, then the matching up rows
__device__ __forceinline__ int block_row_to_global(const JobView& v, int tile, int r) {
  if (v.kind == kJobGateUp) {
    const int u = tile_units(v, tile);
    const int p = v.u0 + tile * 8 + (r < u ? r : r - u);
    return r < u ? p : v.units + p;
  }
  return v.u0 + tile * 16 + r;
}

struct Pipe {
  unsigned char* ring;
  uint64_t* full;    // [kStages] producer -> consumers: the stage's bytes have landed
  uint64_t* empty;   // [kStages] consumers -> producer: every consumer warp is done with the stage
  volatile int* abort_flag;
  int32_t* status;
};

template <bool W_INT8>
__device__ void producer_loop(const MegaParams& p, const Pipe& pipe, int cta, int ncta) {
  constexpr int kElemBytes = W_INT8 ? 1 : 2;
  if ((threadIdx.x & 31) != 0) return;   // one thread issues every copy
  uint64_t policy;
  asm volatile("createpolicy.fractional.L2::evict_first.b64 %0, 1.0;\n" : "=l"(policy));
  int slot = 0;
  uint32_t phase = 0;
  long long issued = 0;
  bool ok = true;
  for (int job = 0; job < p.n_jobs && ok; ++job) {
    const JobView v = job_view<W_INT8>(p.jobs, job, cta, ncta);
    const unsigned char* src = v.wp;
    const int kbytes = v.K * kElemBytes;
    const int kChunkBytes = v.chunk * kElemBytes;
    for (int tg = 0; tg < v.ngroups && ok; ++tg) {
      const int gt = min(GT, v.tiles - tg * GT);
      for (int kc = 0; kc < v.nchunks && ok; ++kc) {
        const int cb = min(kChunkBytes, kbytes - kc * kChunkBytes);
        for (int tile = 0; tile < gt && ok; ++tile) {
          const int rows = tile_rows(v, tg * GT + tile);
          for (int b0 = 0; b0 < cb; b0 += kRowBytes) {
            const uint32_t bytes = (uint32_t)(rows * min(kRowBytes, cb - b0));
            if (!mbar_wait(pipe.empty + slot, phase ^ 1u, pipe.abort_flag, pipe.status)) { ok = false; break; }
            mbar_arrive_expect_tx(pipe.full + slot, bytes);
            bulk_copy(pipe.ring + slot * kStageBytes, src, bytes, pipe.full + slot, policy);
            src += bytes;
            ++issued;
            if (++slot == kStages) { slot = 0; phase ^= 1u; }
          }
        }
      }
    }
  }
  // Nothing of ours may still be in flight when the CTA leaves: wait (bounded) for the stages
  // armed last.  On the normal path the consumers have already waited for all of them.
  const int back = issued < kStages ? (int)issued : kStages;
  for (int i = 0; i < back; ++i) {
    if (--slot < 0) { slot = kStages - 1; phase ^= 1u; }
    const unsigned long long t0 = now_ns();
    while (!mbar_try(pipe.full + slot, phase)) {
      if (now_ns() - t0 > wait_budget(pipe.abort_flag)) { atomicMin(pipe.status, QUASAR_ERR_TIMEOUT); break; }
    }
  }
}

// ---- bounded grid barrier (consumer warps) ---------------------------------------------------
struct GridSync {
  unsigned* counter;
  int32_t* status;
  unsigned ncta;
  unsigned epoch;
  volatile int* abort_flag;  // shared memory
  // The barrier in two halves.  arrive(): this CTA's part of the phase is done and visible.  wait():
  // every CTA's part is.  Between the two a CTA may do whatever neither reads what other CTAs wrote in
  // that phase nor overwrites what they may still be reading.
  __device__ void arrive() {
    cbar();
    ++epoch;
    if (threadIdx.x == 0) {
      // release at GPU scope: everything this CTA wrote before the barrier above (it orders the other
      // threads' writes before this one) is visible to whoever acquires the count
      asm volatile("red.release.gpu.global.add.u32 [%0], %1;\n" ::"l"(counter), "r"(1u) : "memory");
    }
  }
  __device__ bool wait() {
    if (threadIdx.x == 0) {
      const unsigned target = epoch * ncta;
      const unsigned long long t0 = now_ns();
      unsigned polls = 0;
      while (true) {
        unsigned v;
        asm volatile("ld.acquire.gpu.global.u32 %0, [%1];\n" : "=r"(v) : "l"(counter) : "memory");
        if (v >= target) break;
        if ((++polls & 255u) == 0 && (*abort_flag || now_ns() - t0 > wait_budget(abort_flag))) {
          atomicMin(status, QUASAR_ERR_TIMEOUT);
          *abort_flag = 1;
          break;
        }
      }
    }
    cbar();
    return *abort_flag == 0;
  }
  __device__ bool sync() {
    arrive();
    return wait();
  }
};

// ---- operand staging: the <= 8 activation rows of a contraction chunk, in shared memory -------------
// Plain bulk copy global -> shared (both addresses and the size multiples of 16 bytes), counted on `bar`.
__device__ __forceinline__ void bulk_copy_plain(void* smem_dst, const void* gmem_src, uint32_t bytes, uint64_t* bar) {
  asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];\n" ::"r"(
                   (uint32_t)__cvta_generic_to_shared(smem_dst)),
               "l"(gmem_src), "r"(bytes), "r"((uint32_t)__cvta_generic_to_shared(bar))
               : "memory");
}

// Bulk store shared -> global (both addresses and the size multiples of 16 bytes); completion through the
// issuing thread's bulk group.
__device__ __forceinline__ void bulk_store(void* gmem_dst, const void* smem_src, uint32_t bytes) {
  asm volatile("cp.async.bulk.global.shared::cta.bulk_group [%0], [%1], %2;\n" ::"l"(gmem_dst),
               "r"((uint32_t)__cvta_generic_to_shared(smem_src)), "r"(bytes)
               : "memory");
}

// Geometry of an operand buffer: M rows of `len` elements (2 bytes each) at a padded pitch, the chunk of
// the norm gain behind the eighth row.
template <bool W_INT8>
__device__ __forceinline__ int x_pitch(int chunk) { return chunk * 2 + (W_INT8 ? kXPadInt8 : kXPadBf16); }
template <bool W_INT8>
__device__ __forceinline__ int x_buf_bytes(int chunk) { return 8 * x_pitch<W_INT8>(chunk) + chunk * 2; }

// Warp 0 asks for an operand chunk: lane m < M copies row m, lane 8 the norm gain.  A bulk copy keeps the
// whole request in flight at once, which 16-byte loads do not.
template <bool W_INT8>
__device__ __forceinline__ void request_operand(unsigned char* buf, const __nv_bfloat16* src, int ld, int M, int chunk,
                                                int kbase, int len, const __nv_bfloat16* gain, uint64_t* xbar, int lane) {
  const uint32_t cbytes = (uint32_t)len * 2;
  const int pitch = x_pitch<W_INT8>(chunk);
  if (lane == 0) {
    asm volatile("fence.proxy.async.shared::cta;\n" ::: "memory");   // earlier reads / writes of the buffer come first
    mbar_arrive_expect_tx(xbar, (uint32_t)M * cbytes + (gain != nullptr ? cbytes : 0u));
  }
  __syncwarp();
  if (lane < M) bulk_copy_plain(buf + lane * pitch, src + (size_t)lane * ld + kbase, cbytes, xbar);
  if (lane == 8 && gain != nullptr) bulk_copy_plain(buf + 8 * pitch, gain + kbase, cbytes, xbar);
}

// The staged chunk is converted where it lies (a rolled loop: little code, hot after its first turn);
// 32 threads per row, each taking every 32nd 16-byte piece.  Normed GEMMs: h = bf16(x * r * gain), the
// RMSNorm output rounded where the decoder layer rounds it.  int8 weights: h times the row's
// power-of-two scale, as fp16 (exact unless the scaled value falls below the fp16 normal range); the
// scale is folded into rs[row] = r * scale, which commutes with the rounding.  Without a norm rs is the
// scale alone and the gain is one.
template <bool W_INT8>
__device__ __forceinline__ void convert_staged(unsigned char* buf, int M, int chunk, int len, bool has_gain,
                                               const float* rs_row) {
  const int pitch = x_pitch<W_INT8>(chunk);
  const unsigned char* gain = buf + 8 * pitch;
  // the M rows' 16-byte pieces, dealt to all threads in turn (a power-of-two row length keeps the
  // division a shift in the common case; neighbours in a warp take neighbouring pieces)
  const int per_row = len / 8;
#pragma unroll 2
  for (int i = threadIdx.x; i < M * per_row; i += kCT) {
    const int row = i / per_row, c = (i - row * per_row) * 16;
    const float rs = rs_row[row];
    unsigned char* xrow = buf + row * pitch;
    uint4 xv = *reinterpret_cast<const uint4*>(xrow + c);
    uint4 gv = make_uint4(0x3f803f80u, 0x3f803f80u, 0x3f803f80u, 0x3f803f80u);   // bf16 ones
    if (has_gain) gv = *reinterpret_cast<const uint4*>(gain + c);
    uint32_t* w = reinterpret_cast<uint32_t*>(&xv);
    const uint32_t* gw = reinterpret_cast<const uint32_t*>(&gv);
#pragma unroll
    for (int e = 0; e < 4; ++e) {
      // a bf16 is the upper half of an fp32
      const float x0 = __uint_as_float(w[e] << 16), x1 = __uint_as_float(w[e] & 0xffff0000u);
      const float g0 = __uint_as_float(gw[e] << 16), g1 = __uint_as_float(gw[e] & 0xffff0000u);
      const __nv_bfloat162 h = __floats2bfloat162_rn(x0 * rs * g0, x1 * rs * g1);
      if (W_INT8) {
        const uint32_t hb = *reinterpret_cast<const uint32_t*>(&h);
        const __half2 q = __floats2half2_rn(__uint_as_float(hb << 16), __uint_as_float(hb & 0xffff0000u));
        w[e] = *reinterpret_cast<const uint32_t*>(&q);
      } else {
        w[e] = *reinterpret_cast<const uint32_t*>(&h);
      }
    }
    *reinterpret_cast<uint4*>(xrow + c) = xv;
  }
}

// One stage = one block [rows][pb bytes].  MMA row g of the tile is block row ra, MMA row g + 8
// block row rb; the 16-byte pieces of a row are XOR-swizzled by its parity when pb is a multiple
// of 128.  off_a[u] / off_b[u] are this lane's byte offsets for sub-slice u.  `xs` points at this
// lane's share of operand row g for the stage: for sub-slice u the 16 weight bytes of the lane meet 16
// (int8 weights) or 8 (bf16 weights) consecutive operand elements.  The four MMAs of a sub-slice go to
// separate accumulators so that no MMA waits for the one before it.
template <bool W_INT8>
__device__ __forceinline__ void consume_stage(const unsigned char* stage, const unsigned char* xs, const int (&off_a)[kSub],
                                              const int (&off_b)[kSub], unsigned valid_mask, float (&acc)[4][4]) {
  uint4 wa[kSub], wb[kSub], x0[kSub], x1[kSub];
#pragma unroll
  for (int u = 0; u < kSub; ++u) {
    wa[u] = *reinterpret_cast<const uint4*>(stage + off_a[u]);
    wb[u] = *reinterpret_cast<const uint4*>(stage + off_b[u]);
    x0[u] = *reinterpret_cast<const uint4*>(xs + u * (W_INT8 ? 128 : 64));
    if (W_INT8) x1[u] = *reinterpret_cast<const uint4*>(xs + u * 128 + 16);
  }
#pragma unroll
  for (int u = 0; u < kSub; ++u) {
    // Past the end of a short piece the lane reads bytes no copy of this stage has written and operand
    // elements beyond the contraction: both are replaced by zeros (stale bytes may be NaN patterns).
    if (!((valid_mask >> u) & 1u)) {
      x0[u] = make_uint4(0, 0, 0, 0);
      x1[u] = make_uint4(0, 0, 0, 0);
      if (!W_INT8) { wa[u] = make_uint4(0, 0, 0, 0); wb[u] = make_uint4(0, 0, 0, 0); }
    }
    if (W_INT8) {
      uint32_t a0, a1, a2, a3;
      u8x4_to_f16x4(wa[u].x, a0, a2); u8x4_to_f16x4(wb[u].x, a1, a3);
      mma16816_f16(acc[0], a0, a1, a2, a3, x0[u].x, x0[u].y);
      u8x4_to_f16x4(wa[u].y, a0, a2); u8x4_to_f16x4(wb[u].y, a1, a3);
      mma16816_f16(acc[1], a0, a1, a2, a3, x0[u].z, x0[u].w);
      u8x4_to_f16x4(wa[u].z, a0, a2); u8x4_to_f16x4(wb[u].z, a1, a3);
      mma16816_f16(acc[2], a0, a1, a2, a3, x1[u].x, x1[u].y);
      u8x4_to_f16x4(wa[u].w, a0, a2); u8x4_to_f16x4(wb[u].w, a1, a3);
      mma16816_f16(acc[3], a0, a1, a2, a3, x1[u].z, x1[u].w);
    } else {
      mma16816_bf16(acc[2 * (u & 1)], wa[u].x, wb[u].x, wa[u].y, wb[u].y, x0[u].x, x0[u].y);
      mma16816_bf16(acc[2 * (u & 1) + 1], wa[u].z, wb[u].z, wa[u].w, wb[u].w, x0[u].z, x0[u].w);
    }
  }
}

// byte offset, inside a block of pitch pb, of the 16 bytes lane (warp, t) reads from block row r in sub-slice u
__device__ __forceinline__ int block_offset(int r, int pb, int warp, int u, int t) {
  int chunk = (warp * kWarpBytes + u * 64) / 16 + t;
  if ((pb & 127) == 0) chunk ^= (r & 1) << 2;
  return r * pb + chunk * 16;
}

// ---- one GEMM phase (consumer warps) -------------------------------------------------------------
template <bool W_INT8>
struct GemmPhase {
  static constexpr int kElemBytes = W_INT8 ? 1 : 2;
  static constexpr int kItems = GT * 128 / kCT;   // epilogue elements per consumer thread and tile group
  static_assert(kItems * kCT == GT * 128 && kCT % 128 == 0, "epilogue elements divide evenly; a thread keeps its operand row");

  __device__ __forceinline__ static bool run(const MegaParams& p, int job, const Pipe& pipe, int& slot_io,
                                             uint32_t& phase_io, float* red, float* misc, unsigned char* x_s, uint64_t* xbar,
                                             uint32_t& xphase, int cta, int ncta, GridSync& gs) {
    int slot = slot_io;
    uint32_t phase = phase_io;
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31, g = lane >> 2, t = lane & 3;
    // The phase's descriptor was fetched into shared memory during the phase before (a load from global
    // memory here would be the first thing every warp waits for); thread 0 now fetches the next one into
    // the other slot, which nobody has read since the phase before last.
    MegaJob* job_s = reinterpret_cast<MegaJob*>(misc + kMiscJob);
    const MegaJob jb = job_s[job & 1];
    if (threadIdx.x == 0 && job + 1 < p.n_jobs) job_s[(job + 1) & 1] = p.jobs[job + 1];
    const JobView v = job_view_of<W_INT8>(jb, cta, ncta);
    const int M = p.M;
    const bool normed = jb.gain != nullptr;
    const bool residual = jb.kind == kJobO || jb.kind == kJobDown;
    const __nv_bfloat16* xsrc = jb.kind == kJobO ? p.attn : (jb.kind == kJobDown ? p.act : p.x);
    const int ld = jb.K;
    // int8 weights: the operands of the o and down projections also exist as fp16, exactly what the
    // conversion below would make of them as long as no row needs a scale (no element beyond 2^15).
    // The phase asks for that copy first and falls back to the bf16 tensor if a row maximum says otherwise.
    const bool has16 = W_INT8 && (jb.kind == kJobO || jb.kind == kJobDown);
    const __nv_bfloat16* xsrc16 = reinterpret_cast<const __nv_bfloat16*>(jb.kind == kJobO ? p.attn16 : p.act16);
    bool direct = has16;   // the staged chunk needs no conversion

    // The operand of the first chunk and the per-row factors, all in ONE round trip to L2: the
    // loads of the operand, of the gains and of the statistics are issued together.  Normed GEMMs:
    // the RMSNorm factor comes from the per-CTA sums of squares that the phase which wrote x left
    // behind (each warp adds its share of the CTAs, the shares meet in shared memory: a fixed order);
    // the fp16 scale is the job's static one (|h| <= sqrt(K) * max|gain|).  Other GEMMs with int8
    // weights: a power-of-two scale from the row maximum gathered while the operand was written.
    bool have_x = false, first = true;
    bool requested = false;   // the next chunk's copy is already in flight
    int xb = 0;               // operand buffer in use (a long contraction alternates between two)
    const int xpitch = x_pitch<W_INT8>(v.chunk);
    const int xbuf_bytes = x_buf_bytes<W_INT8>(v.chunk);
    float ss_run = 0.f;   // threads 0..7 (o / down): sum of squares of the row of x this CTA has written
    float best = -INFINITY;   // LM head: this thread's running arg-max over the elements it finishes
    int best_i = 0x7fffffff;

    // The caller has arrived at the grid barrier that ends the phase before; this phase waits for it only
    // where it first needs that phase's results (below, after the loads that do not depend on them).
    if (v.ngroups == 0 && !gs.wait()) return false;
    for (int tg = 0; tg < v.ngroups; ++tg) {
      const int gt = min(GT, v.tiles - tg * GT);
      // The elements this thread finishes in the group's epilogue (element e = thread + it * kCT of the
      // group's GT x 16 x 8); their step sizes and residuals are requested now so that the epilogue
      // does not wait for them.
      float d0[kItems], d1[kItems], resid[kItems];
#pragma unroll
      for (int it = 0; it < kItems; ++it) {
        const EpiItem ei = epi_item(jb, v, tg, gt, M, it);
        d0[it] = d1[it] = 1.f;
        resid[it] = 0.f;
        if (ei.ok) {
          if (jb.delta != nullptr) {
            d0[it] = ld_early_f32(jb.delta + ei.unit);
            if (jb.kind == kJobGateUp) d1[it] = ld_early_f32(jb.delta + v.units + ei.unit);
          }
          if (residual) resid[it] = ld_early_bf16_cg(p.x + (size_t)ei.col * jb.N + ei.unit);
        }
      }
      if (tg == 0) {
        // (the step sizes and residuals above do not depend on the phase before: the residual stream was
        // last written two phases ago)  Now the operand: every CTA's part of it must be there.
        if (!gs.wait()) return false;
        // Its first chunk is asked for at once: the round trip to L2 is the longest wait of the prologue.
        // (Every warp is past its last use of the buffer's other tenants: the epilogue and the attention
        // phase end in a CTA barrier.)
        if (warp == 0)
          request_operand<W_INT8>(x_s, direct ? xsrc16 : xsrc, ld, M, v.chunk, 0, min(v.chunk, jb.K), jb.gain, xbar, lane);
        requested = true;
      }

      // Accumulators live for one tile and one chunk; each warp then parks them in its own part of
      // `red` (summing over the chunks of a long contraction), where the epilogue adds the warps up.
      for (int kc = 0; kc < v.nchunks; ++kc) {
        if (!have_x) {
          // every warp is past its last use of the buffer's other tenants (epilogue / attention end in a CTA barrier)
          if (warp == 0 && !requested)
            request_operand<W_INT8>(x_s + xb * xbuf_bytes, direct ? xsrc16 : xsrc, ld, M, v.chunk, kc * v.chunk,
                                    min(v.chunk, jb.K - kc * v.chunk), jb.gain, xbar, lane);
          requested = false;
          bool again = false;   // the fp16 copy was asked for, but a row needs a scale
          if (first) {   // the row factors ride on the same round trip as the first chunk's loads
            first = false;
            float rnorm = 1.f, xscale = 1.f, inv = 1.f;
            if (normed) {
              const int per_warp = (ncta + NW - 1) / NW;
              const int c_end = min(ncta, (warp + 1) * per_warp);
              float ss = 0.f;
              for (int c = warp * per_warp + t; c < c_end; c += 4) ss += __ldcg(p.ss_part + c * 8 + g);
              ss += __shfl_xor_sync(0xffffffffu, ss, 1);
              ss += __shfl_xor_sync(0xffffffffu, ss, 2);
              if (t == 0) misc[kMiscRowSum + warp * 8 + g] = ss;
              cbar();
              float tot = 0.f;
#pragma unroll
              for (int w = 0; w < NW; ++w) tot += misc[kMiscRowSum + w * 8 + g];
              rnorm = 1.0f / sqrtf(tot / (float)jb.K + p.rms_eps);
              if (W_INT8) { xscale = jb.xscale; inv = 1.0f / xscale; }
            } else if (W_INT8) {
              const float mx = __uint_as_float(__ldcg(p.amax_buf + job * 8 + g));
              if (mx > 32768.f && mx < 3.0e38f) {
                int e;
                (void)frexpf(mx, &e);               // mx = f * 2^e, f in [0.5, 1)
                xscale = ldexpf(1.f, 15 - e);       // scaled row maximum <= 2^15
                inv = ldexpf(1.f, e - 15);
              }
              if (has16) {   // the same answer in every warp: all read the same eight maxima
                float top = mx;   // (NaN compares false: such a row goes the converting way below)
                top = fmaxf(top, __shfl_xor_sync(0xffffffffu, top, 4));
                top = fmaxf(top, __shfl_xor_sync(0xffffffffu, top, 8));
                top = fmaxf(top, __shfl_xor_sync(0xffffffffu, top, 16));
                direct = __all_sync(0xffffffffu, mx <= 32768.f) && top <= 32768.f;
                again = !direct;
              }
            }
            if (warp == 0 && t == 0) {
              misc[kMiscRs + g] = rnorm * xscale;   // conversion factor of operand row g
              misc[kMiscInvScale + g] = inv;
            }   // read by the conversion and in the epilogues, behind a CTA barrier
          }
          {
            int got = 1;
            if (lane == 0) got = mbar_wait(xbar, xphase, pipe.abort_flag, pipe.status) ? 1 : 0;
            got = __shfl_sync(0xffffffffu, got, 0);
            if (!got) return false;
            xphase ^= 1u;
          }
          if (again) {   // rare: fetch the chunk once more, from the bf16 tensor
            cbar();      // every warp has seen the first copy land
            if (warp == 0)
              request_operand<W_INT8>(x_s + xb * xbuf_bytes, xsrc, ld, M, v.chunk, kc * v.chunk,
                                      min(v.chunk, jb.K - kc * v.chunk), jb.gain, xbar, lane);
            int got = 1;
            if (lane == 0) got = mbar_wait(xbar, xphase, pipe.abort_flag, pipe.status) ? 1 : 0;
            got = __shfl_sync(0xffffffffu, got, 0);
            if (!got) return false;
            xphase ^= 1u;
          }
          if (!direct && (W_INT8 || normed)) {
            cbar();   // the rows' factors are published
            convert_staged<W_INT8>(x_s + xb * xbuf_bytes, M, v.chunk, min(v.chunk, jb.K - kc * v.chunk), normed, misc + kMiscRs);
          }
          cbar();   // the chunk is ready; every warp is past the tiles of the chunk before it
          if (v.nchunks > 1 && (kc + 1 < v.nchunks || tg + 1 < v.ngroups)) {
            // a long contraction reloads its chunks for every tile group: the next one lands in the
            // other buffer while this one is multiplied
            const int nk = kc + 1 < v.nchunks ? kc + 1 : 0;
            if (warp == 0)
              request_operand<W_INT8>(x_s + (xb ^ 1) * xbuf_bytes, direct ? xsrc16 : xsrc, ld, M, v.chunk, nk * v.chunk,
                                      min(v.chunk, jb.K - nk * v.chunk), jb.gain, xbar, lane);
            requested = true;
          }
        }
        const int cb = min(v.chunk, jb.K - kc * v.chunk) * kElemBytes;   // bytes of a weight row in this chunk
        const int nst = (cb + kRowBytes - 1) / kRowBytes;                 // stages per tile
        const int pb_last = cb - (nst - 1) * kRowBytes;                   // bytes of a row's last piece
        // this lane's share of operand row g: the elements that meet the warp's weight bytes, stage by stage
        const unsigned char* xlane = x_s + xb * xbuf_bytes + g * xpitch + (warp * kWarpBytes + t * 16) * (2 / kElemBytes);
        // Block rows behind MMA rows g and g + 8: rows g and g + 8 of the stage (rows past a tile stay inside
        // the stage and feed accumulator rows that are never stored); only a gate/up tile with fewer than 8
        // pairs keeps its up rows elsewhere (right behind its gate rows).  This lane's byte offsets in a
        // stage of full pieces and in the stage of the rows' last pieces are the same for every such tile.
        int oa_full[kSub], ob_full[kSub], oa_last[kSub], ob_last[kSub];
        unsigned mask_last = 0;
#pragma unroll
        for (int u = 0; u < kSub; ++u) {
          // a lane past the end of a short piece reads inside the stage (offset < 16 KB) but not its own data
          const bool lane_valid = warp * kWarpBytes + u * 64 + t * 16 < pb_last;
          mask_last |= (lane_valid ? 1u : 0u) << u;
          oa_full[u] = block_offset(g, kRowBytes, warp, u, t);
          ob_full[u] = block_offset(g + 8, kRowBytes, warp, u, t);
          oa_last[u] = lane_valid ? block_offset(g, pb_last, warp, u, t) : 0;
          ob_last[u] = lane_valid ? block_offset(g + 8, pb_last, warp, u, t) : 0;
        }
#pragma unroll 1
        for (int tile = 0; tile < gt; ++tile) {
          if (v.kind == kJobGateUp && tile_units(v, tg * GT + tile) != 8) {   // the short last tile of a gate/up range
            const int rb = tile_units(v, tg * GT + tile) + g;
#pragma unroll
            for (int u = 0; u < kSub; ++u) {
              ob_full[u] = block_offset(rb, kRowBytes, warp, u, t);
              ob_last[u] = ((mask_last >> u) & 1u) ? block_offset(rb, pb_last, warp, u, t) : 0;
            }
          }
          float ch[4][4];
#pragma unroll
          for (int i = 0; i < 4; ++i) ch[i][0] = ch[i][1] = ch[i][2] = ch[i][3] = 0.f;
#pragma unroll 1
          for (int st = 0; st < nst; ++st) {   // rolled: the stage's code stays in the instruction cache
            const bool last = st == nst - 1;
            int oa[kSub], ob[kSub];
#pragma unroll
            for (int u = 0; u < kSub; ++u) {
              oa[u] = last ? oa_last[u] : oa_full[u];
              ob[u] = last ? ob_last[u] : ob_full[u];
            }
            const unsigned valid_mask = last ? mask_last : (1u << kSub) - 1u;
            // every lane tests the stage's barrier itself (one instruction per warp, no broadcast afterwards)
            if (!__all_sync(0xffffffffu, mbar_wait(pipe.full + slot, phase, pipe.abort_flag, pipe.status))) return false;   // the warp leaves together
            consume_stage<W_INT8>(pipe.ring + slot * kStageBytes, xlane + st * (kRowBytes * 2 / kElemBytes), oa, ob, valid_mask, ch);
            __syncwarp();
            if (lane == 0) mbar_arrive(pipe.empty + slot);
            if (++slot == kStages) { slot = 0; phase ^= 1u; }
          }
          float* r = red + ((warp * GT + tile) * 16) * 8;
          float2 lo = make_float2((ch[0][0] + ch[1][0]) + (ch[2][0] + ch[3][0]), (ch[0][1] + ch[1][1]) + (ch[2][1] + ch[3][1]));
          float2 hi = make_float2((ch[0][2] + ch[1][2]) + (ch[2][2] + ch[3][2]), (ch[0][3] + ch[1][3]) + (ch[2][3] + ch[3][3]));
          float2* plo = reinterpret_cast<float2*>(r + g * 8 + 2 * t);
          float2* phi = reinterpret_cast<float2*>(r + (g + 8) * 8 + 2 * t);
          if (kc > 0) {   // only this thread touches these two slots
            const float2 a = *plo, b = *phi;
            lo.x += a.x; lo.y += a.y; hi.x += b.x; hi.y += b.y;
          }
          *plo = lo;
          *phi = hi;
        }
        if (v.nchunks > 1) xb ^= 1;   // the next chunk is (or will be) in the other buffer
        else have_x = true;           // a short contraction keeps its operand for every tile group
      }
      // ---- cross-warp reduction in a fixed order, then the fused epilogue ----
      cbar();
#pragma unroll 1
      for (int it = 0; it < kItems; ++it) {   // rolled: the epilogue's code exists once
        const EpiItem ei = epi_item(jb, v, tg, gt, M, it);
        float e0 = d0[0], e1 = d1[0], er = resid[0];
#pragma unroll
        for (int j = 1; j < kItems; ++j) {
          if (it == j) { e0 = d0[j]; e1 = d1[j]; er = resid[j]; }
        }
        epilogue(p, jb, v, job, ei, e0, e1, er, best, best_i, red, misc);
      }
      cbar();
      if (residual && threadIdx.x < 8) {   // fixed order: tiles of the group, groups of the phase
        for (int tile = 0; tile < gt; ++tile) ss_run += misc[kMiscPart + tile * 8 + threadIdx.x];
      }
    }
    if (residual && threadIdx.x < 8) p.ss_part[cta * 8 + threadIdx.x] = ss_run;
    if (jb.kind == kJobLm) finish_argmax(best, best_i, misc);
    slot_io = slot;
    phase_io = phase;
    return true;
  }

  struct EpiItem {
    int tile, row, col, unit;   // tile in the group, MMA row, operand row, output channel (or gate/up pair)
    bool ok;
  };
  __device__ __forceinline__ static EpiItem epi_item(const MegaJob& jb, const JobView& v, int tg, int gt, int M, int it) {
    const int e = (int)threadIdx.x + it * kCT;
    EpiItem ei;
    ei.tile = jb.kind == kJobGateUp ? e >> 6 : e >> 7;
    ei.col = jb.kind == kJobGateUp ? (e >> 3) & 7 : (e >> 4) & 7;
    ei.row = jb.kind == kJobGateUp ? e & 7 : e & 15;
    ei.unit = v.u0 + (tg * GT + ei.tile) * v.rows_per_tile + ei.row;
    ei.ok = ei.tile < gt && ei.unit < v.u1 && ei.col < M;
    return ei;
  }

  __device__ __forceinline__ static float reduce_at(const float* red, int tile, int row, int col) {
    float s = 0.f;
#pragma unroll
    for (int w = 0; w < NW; ++w) s += red[((w * GT + tile) * 16 + row) * 8 + col];
    return s;
  }

  // One output element per thread: sum the warps' partials, apply the step size (and the operand's
  // scale), then what the step of the pass asks for.
  __device__ __forceinline__ static void epilogue(const MegaParams& p, const MegaJob& jb, const JobView& v, int job,
                                                  const EpiItem& ei, float d0, float d1, float resid, float& best,
                                                  int& best_i, const float* red, float* misc) {
    const int lane = threadIdx.x & 31;
    const bool ok = ei.ok;
    const int tile = ei.tile, row = ei.row, col = ei.col, unit_idx = ei.unit;
    const float unit = W_INT8 ? misc[kMiscInvScale + col] : 1.f;
    if (jb.kind == kJobGateUp) {
      // SwiGLU: act = silu(gate) * up, gate and up rounded to bf16 first (they are tensors of the layer)
      float a = 0.f;
      if (ok) {
        const float gate = bf16_round_f(reduce_at(red, tile, row, col) * unit * d0);
        const float up = bf16_round_f(reduce_at(red, tile, row + 8, col) * unit * d1);
        const __nv_bfloat16 av = __float2bfloat16_rn(gate / (1.0f + expf(-gate)) * up);
        p.act[(size_t)col * v.units + unit_idx] = av;
        if (W_INT8) p.act16[(size_t)col * v.units + unit_idx] = __half_as_ushort(__float2half_rn(__bfloat162float(av)));
        a = fabsf(__bfloat162float(av));
      }
      if (W_INT8) {   // row maximum of the next GEMM's operand (8 consecutive lanes share a row)
        a = fmaxf(a, __shfl_xor_sync(0xffffffffu, a, 1));
        a = fmaxf(a, __shfl_xor_sync(0xffffffffu, a, 2));
        a = fmaxf(a, __shfl_xor_sync(0xffffffffu, a, 4));
        if ((lane & 7) == 0 && a > 0.f) atomicMax(p.amax_buf + (job + 1) * 8 + col, __float_as_uint(a));
      }
      return;
    }
    float sq = 0.f;
    if (ok) {
      const float val = reduce_at(red, tile, row, col) * unit * d0;
      const size_t idx = (size_t)col * jb.N + unit_idx;
      if (jb.kind == kJobQkv) {
        p.qkv[idx] = __float2bfloat16_rn(val);
      } else if (jb.kind == kJobLm) {
        if (p.logits) p.logits[idx] = val;
        // a thread's channels only grow from group to group: on equal values the earlier, lower one stays
        if (val > best) { best = val; best_i = unit_idx; }
      } else {  // o / down: residual add into the stream
        const __nv_bfloat16 xn = __float2bfloat16_rn(bf16_round_f(val) + resid);
        p.x[idx] = xn;
        const float xf = __bfloat162float(xn);
        sq = xf * xf;
      }
    }
    if (jb.kind == kJobO || jb.kind == kJobDown) {
      // sum of squares of what this CTA adds to each row of x (16 consecutive lanes share tile and row)
#pragma unroll
      for (int o = 8; o > 0; o >>= 1) sq += __shfl_xor_sync(0xffffffffu, sq, o);
      if ((lane & 15) == 0) misc[kMiscPart + tile * 8 + col] = sq;
    }
  }

  // End of the LM head: the CTA's arg-max per operand row from its threads' running ones (lowest
  // channel on ties).  16 consecutive lanes share a row, as do the threads 128 apart.
  __device__ __forceinline__ static void finish_argmax(float best, int best_i, float* misc) {
#pragma unroll
    for (int o = 8; o > 0; o >>= 1) {
      const float ob = __shfl_xor_sync(0xffffffffu, best, o);
      const int oi = __shfl_xor_sync(0xffffffffu, best_i, o);
      if (ob > best || (ob == best && oi < best_i)) { best = ob; best_i = oi; }
    }
    float* cand_v = misc + kMiscCand;
    int* cand_i = reinterpret_cast<int*>(misc + kMiscCand + 64);
    if ((threadIdx.x & 15) == 0) {
      cand_v[threadIdx.x >> 4] = best;
      cand_i[threadIdx.x >> 4] = best_i;
    }
    cbar();
    if (threadIdx.x < 8) {
      float bv = -INFINITY;
      int bi = 0x7fffffff;
      for (int q = threadIdx.x; q < kCT / 16; q += 8) {
        const float ov = cand_v[q];
        const int oi = cand_i[q];
        if (ov > bv || (ov == bv && oi < bi)) { bv = ov; bi = oi; }
      }
      misc[kMiscRunV + threadIdx.x] = bv;
      reinterpret_cast<int*>(misc + kMiscRunI)[threadIdx.x] = bi;
    }
  }
};

// ---- block bookkeeping + embedding gather (phase 0) -------------------------------------------
__device__ void prep_phase(const MegaParams& p, float* misc, int cta, int ncta) {
  // one thread per sequence validates the block and derives ancestor masks / depths
  if (cta == 0 && (int)threadIdx.x < p.B) {
    const int b = threadIdx.x;
    const int T = p.block_len[b], P = p.seq_len[b];
    int err = 0;
    if (T < 1 || T > p.T_max || P < 0) err = QUASAR_ERR_INVALID_ARG;
    else if (P + T > p.s_max) err = QUASAR_ERR_CAPACITY;
    if (!err) {
      for (int i = 0; i < T; ++i) {
        const int tok = p.tokens[b * p.T_max + i];
        if (tok < 0 || tok >= p.vocab) err = QUASAR_ERR_TOKEN;
        const int par = p.parents ? p.parents[b * p.T_max + i] : i - 1;
        if ((i == 0 && par != -1) || (i > 0 && (par < 0 || par >= i))) err = QUASAR_ERR_TREE;
        if (err) break;
        uint64_t m = 1ull << i;
        int d = 0;
        if (i > 0) { m |= p.bi.anc[b * p.T_max + par]; d = p.bi.depth[b * p.T_max + par] + 1; }
        p.bi.anc[b * p.T_max + i] = m;
        p.bi.depth[b * p.T_max + i] = d;
      }
    }
    for (int i = (err ? 0 : T); i < p.T_max; ++i) { p.bi.anc[b * p.T_max + i] = 0; p.bi.depth[b * p.T_max + i] = 0; }
    p.bi.valid[b] = err ? 0 : 1;
    if (err) atomicMin(p.status, err);
  }
  // row maxima of the un-normed GEMM operands start at zero (gathered with atomicMax during the pass)
  for (int i = cta * kCT + threadIdx.x; i < p.n_jobs * 8; i += ncta * kCT) p.amax_buf[i] = 0u;
  for (int i = cta * kCT + threadIdx.x; i < p.L * p.B * p.Hkv; i += ncta * kCT) p.attn_count[i] = 0u;
  // Embedding rows: CTA m gathers row m and leaves its sum of squares for the first RMSNorm; every
  // CTA leaves a (possibly zero) entry per row, the layout the later phases use too.
  float* wsum = misc + kMiscRowSum;
  const int m = cta;   // the grid has at least 8 CTAs
  float ss = 0.f;
  if (m < p.M) {
    const int tok = p.tokens[m];
    const bool ok = tok >= 0 && tok < p.vocab;
    for (int c = threadIdx.x; c < p.H / 8; c += kCT) {
      uint4 v = make_uint4(0, 0, 0, 0);
      if (ok) v = __ldg(reinterpret_cast<const uint4*>(p.embed + (size_t)tok * p.H) + c);
      reinterpret_cast<uint4*>(p.x + (size_t)m * p.H)[c] = v;
      const __nv_bfloat162* h = reinterpret_cast<const __nv_bfloat162*>(&v);
#pragma unroll
      for (int e = 0; e < 4; ++e) {
        const float2 f = __bfloat1622float2(h[e]);
        ss += f.x * f.x + f.y * f.y;
      }
    }
  }
  ss = warp_sum(ss);
  if ((threadIdx.x & 31) == 0) wsum[threadIdx.x >> 5] = ss;
  cbar();
  if (threadIdx.x < 8) {
    float tot = 0.f;
    if ((int)threadIdx.x == m && m < p.M) {
      for (int w = 0; w < NW; ++w) tot += wsum[w];
    }
    p.ss_part[cta * 8 + threadIdx.x] = tot;
  }
}

// ---- attention phase: QK-RMSNorm + RoPE + KV append + split-KV partials -------------------------
// kP consecutive bf16 (kP = 4 or 8) from / to 8- or 16-byte aligned memory, as floats
template <int kP>
__device__ __forceinline__ void load_bf16_vec(float (&f)[kP], const __nv_bfloat16* src, bool through_l2) {
  uint32_t w[kP / 2];
  if constexpr (kP == 8) {
    const uint4 v = through_l2 ? __ldcg(reinterpret_cast<const uint4*>(src)) : __ldg(reinterpret_cast<const uint4*>(src));
    w[0] = v.x; w[1] = v.y; w[2] = v.z; w[3] = v.w;
  } else {
    const uint2 v = through_l2 ? __ldcg(reinterpret_cast<const uint2*>(src)) : __ldg(reinterpret_cast<const uint2*>(src));
    w[0] = v.x; w[1] = v.y;
  }
#pragma unroll
  for (int i = 0; i < kP / 2; ++i) {
    f[2 * i] = __uint_as_float(w[i] << 16);
    f[2 * i + 1] = __uint_as_float(w[i] & 0xffff0000u);
  }
}
template <int kP>
__device__ __forceinline__ void store_bf16_vec(__nv_bfloat16* dst, const float (&f)[kP]) {
  uint32_t w[kP / 2];
#pragma unroll
  for (int i = 0; i < kP / 2; ++i) w[i] = pack_bf16(f[2 * i], f[2 * i + 1]);
  if constexpr (kP == 8) *reinterpret_cast<uint4*>(dst) = make_uint4(w[0], w[1], w[2], w[3]);
  else *reinterpret_cast<uint2*>(dst) = make_uint2(w[0], w[1]);
}

__device__ __forceinline__ void cp_async16(void* smem, const void* gmem) {
  asm volatile("cp.async.cg.shared.global [%0], [%1], 16;\n" ::"r"((uint32_t)__cvta_generic_to_shared(smem)), "l"(gmem)
               : "memory");
}

// The attention work items: (sequence, kv head, chunk of kKeyTile keys), item = (b * Hkv + hk) * nchunk + c.
// Called before the grid barrier that ends the qkv GEMM: starts copying the part of this CTA's first
// K/V tile that is already in the cache (keys before seq_len), so that the copy's latency hides
// behind the barrier.  The tiles alias the GEMM's reduction buffer, which is free by then.
template <int D>
__device__ __forceinline__ void attention_prefetch(const MegaParams& p, int layer, __nv_bfloat16* k_s,
                                                   __nv_bfloat16* v_s, int cta) {
  constexpr int kStride = D + 8;
  const int n_items = p.B * p.Hkv * p.attn_nchunk;
  if (cta < n_items) {
    const int c = cta % p.attn_nchunk;
    const int hk = (cta / p.attn_nchunk) % p.Hkv;
    const int b = cta / (p.attn_nchunk * p.Hkv);
    if (p.bi.valid[b]) {
      const int P = p.seq_len[b];
      const int key_begin = c * kKeyTile;
      const int rows = min(kKeyTile, P - key_begin);
      const size_t layer_stride = (size_t)p.kv_batch * p.Hkv * (size_t)p.s_max * D;
      const size_t head_off = (size_t)layer * layer_stride + ((size_t)b * p.Hkv + hk) * (size_t)p.s_max * D;
      const __nv_bfloat16* kbase = p.k_cache + head_off + (size_t)key_begin * D;
      const __nv_bfloat16* vbase = p.v_cache + head_off + (size_t)key_begin * D;
      for (int i = threadIdx.x; i < rows * (D / 8); i += kCT) {
        const int key = i / (D / 8), ch = i % (D / 8);
        cp_async16(k_s + key * kStride + ch * 8, kbase + (size_t)key * D + ch * 8);
        cp_async16(v_s + key * kStride + ch * 8, vbase + (size_t)key * D + ch * 8);
      }
    }
  }
  asm volatile("cp.async.commit_group;\n" ::: "memory");
}

template <int D>
__device__ __noinline__ void attention_phase(const MegaParams& p, int layer, bool want_amax, __nv_bfloat16* k_s,
                                             __nv_bfloat16* v_s, __nv_bfloat16* q_s, float* misc, uint64_t* xbar,
                                             uint32_t& xphase, uint32_t& xphase2, int cta, int ncta) {
  float* o_s = reinterpret_cast<float*>(reinterpret_cast<unsigned char*>(k_s) + 2 * kKvTileBytes + kQTileBytes);
  float* ml_s = o_s + kMaxRowsAttn * 128;
  volatile int* abort_flag = reinterpret_cast<volatile int*>(misc + kMiscAbort);
  constexpr int kStride = D + 8;
  constexpr int kDSteps = D / 16;
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31, g = lane >> 2, t = lane & 3;
  const int G = p.Hq / p.Hkv;
  const int qkv_w = (p.Hq + 2 * p.Hkv) * D;
  const MegaLayer ly = p.layers[layer];
  const size_t layer_stride = (size_t)p.kv_batch * p.Hkv * (size_t)p.s_max * D;
  __nv_bfloat16* kc_l = p.k_cache + (size_t)layer * layer_stride;
  __nv_bfloat16* vc_l = p.v_cache + (size_t)layer * layer_stride;
  const int n_items = p.B * p.Hkv * p.attn_nchunk;
  int* last_flag = reinterpret_cast<int*>(misc + kMiscFlag);

  // rows that take no part (beyond a block's length, or of a skipped sequence) give zero attention output
  for (int m = cta; m < p.M; m += ncta) {
    const int b = m / p.T_max, i = m % p.T_max;
    if (!p.bi.valid[b] || i >= p.block_len[b]) {
      uint4* dst = reinterpret_cast<uint4*>(p.attn + (size_t)m * p.Hq * D);
      uint4* dst16 = reinterpret_cast<uint4*>(p.attn16 + (size_t)m * p.Hq * D);
      for (int j = threadIdx.x; j < p.Hq * D / 8; j += kCT) {
        dst[j] = make_uint4(0, 0, 0, 0);
        dst16[j] = make_uint4(0, 0, 0, 0);
      }
    }
  }

  for (int item = cta; item < n_items; item += ncta) {
    const int c = item % p.attn_nchunk;
    const int hk = (item / p.attn_nchunk) % p.Hkv;
    const int b = item / (p.attn_nchunk * p.Hkv);
    const bool prefetched = item == cta;   // attention_prefetch has started the cached rows of this tile
    if (!p.bi.valid[b]) continue;
    const int T = p.block_len[b], P = p.seq_len[b];
    const int Lk = P + T;
    const int key_begin = c * kKeyTile, key_end = min(Lk, key_begin + kKeyTile);
    if (key_begin >= key_end) continue;
    __nv_bfloat16* kbase = kc_l + ((size_t)b * p.Hkv + hk) * (size_t)p.s_max * D;
    __nv_bfloat16* vbase = vc_l + ((size_t)b * p.Hkv + hk) * (size_t)p.s_max * D;
    const int R = G * T;
    cbar();  // shared tiles of the previous item are no longer read

    // (a) rotate this kv head's query rows into shared memory; the item that owns a block row's
    //     cache slot also rotates its K row and stores K and V there
    // A quarter of a warp per head vector (four vectors per warp at a time, one code path): lane q8 owns
    // the rotation pairs (d, d + D/2) for d = kP q8 .. kP q8 + kP - 1.
    {
      constexpr int kP = D / 16;
      const int q8 = lane & 7, d0 = q8 * kP;
#pragma unroll 1
      for (int ub = warp * 4; ub < R + T; ub += NW * 4) {
        const int u = ub + (lane >> 3);
        int kind = 0;   // 0 nothing, 1 query vector, 2 key vector (with its value row)
        int m = 0, slot = 0;
        const __nv_bfloat16* src = p.qkv;
        if (u < R) {
          kind = 1;
          m = b * p.T_max + u / G;
          src = p.qkv + (size_t)m * qkv_w + (size_t)(hk * G + (u % G)) * D;
        } else if (u < R + T) {
          slot = P + (u - R);
          if (slot >= key_begin && slot < key_end) {
            kind = 2;
            m = b * p.T_max + (u - R);
            src = p.qkv + (size_t)m * qkv_w + (size_t)(p.Hq + hk) * D;
          }
        }
        const __nv_bfloat16* gain = kind == 2 ? ly.k_norm : ly.q_norm;
        float lo[kP], hi[kP], glo[kP], ghi[kP];
        float4 cs[kP / 2];
        uint4 vrow[kP / 4];
#pragma unroll
        for (int i = 0; i < kP; ++i) { lo[i] = hi[i] = 0.f; glo[i] = ghi[i] = 1.f; }
        if (kind != 0) {   // every load of the vector before any use
          load_bf16_vec<kP>(lo, src + d0, true);
          load_bf16_vec<kP>(hi, src + D / 2 + d0, true);
          const float4* cp = reinterpret_cast<const float4*>(p.rope_table + (size_t)(P + p.bi.depth[m]) * (D / 2) + d0);
#pragma unroll
          for (int i = 0; i < kP / 2; ++i) cs[i] = __ldg(cp + i);
          if (gain != nullptr) {
            load_bf16_vec<kP>(glo, gain + d0, false);
            load_bf16_vec<kP>(ghi, gain + D / 2 + d0, false);
          }
          if (kind == 2) {
            const uint4* vsrc = reinterpret_cast<const uint4*>(p.qkv + (size_t)m * qkv_w + (size_t)(p.Hq + p.Hkv + hk) * D) + q8 * (kP / 4);
#pragma unroll
            for (int i = 0; i < kP / 4; ++i) vrow[i] = __ldcg(vsrc + i);
          }
        }
        if (ly.q_norm != nullptr) {   // QK-RMSNorm (a model either has both gains or none)
          float ss = 0.f;
#pragma unroll
          for (int i = 0; i < kP; ++i) ss += lo[i] * lo[i] + hi[i] * hi[i];
          ss += __shfl_xor_sync(0xffffffffu, ss, 1);
          ss += __shfl_xor_sync(0xffffffffu, ss, 2);
          ss += __shfl_xor_sync(0xffffffffu, ss, 4);
          const float rn = 1.0f / sqrtf(ss / (float)D + p.rms_eps);
#pragma unroll
          for (int i = 0; i < kP; ++i) { lo[i] = lo[i] * rn * glo[i]; hi[i] = hi[i] * rn * ghi[i]; }
        }
        if (kind != 0) {
          float olo[kP], ohi[kP];
#pragma unroll
          for (int i = 0; i < kP; ++i) {
            const float c = (i & 1) ? cs[i / 2].z : cs[i / 2].x, sn = (i & 1) ? cs[i / 2].w : cs[i / 2].y;
            olo[i] = lo[i] * c - hi[i] * sn;
            ohi[i] = hi[i] * c + lo[i] * sn;
          }
          __nv_bfloat16* dst = kind == 1 ? q_s + u * kStride : kbase + (size_t)slot * D;
          store_bf16_vec<kP>(dst + d0, olo);
          store_bf16_vec<kP>(dst + D / 2 + d0, ohi);
          if (kind == 2) {
            uint4* vdst = reinterpret_cast<uint4*>(vbase + (size_t)slot * D) + q8 * (kP / 4);
#pragma unroll
            for (int i = 0; i < kP / 4; ++i) vdst[i] = vrow[i];
          }
        }
      }
    }
    cbar();  // block-level visibility of the K/V rows just stored and of q_s
    // (b) stage the K / V tile (zero beyond the end of the sequence); cached rows of a prefetched
    //     tile are already on their way
    const int first_row = prefetched ? max(0, min(kKeyTile, P - key_begin)) : 0;
    for (int i = first_row * (D / 8) + threadIdx.x; i < kKeyTile * (D / 8); i += kCT) {
      const int key = i / (D / 8), ch = i % (D / 8);
      uint4 kv4 = make_uint4(0, 0, 0, 0), vv4 = make_uint4(0, 0, 0, 0);
      if (key_begin + key < key_end) {
        kv4 = __ldcg(reinterpret_cast<const uint4*>(kbase + (size_t)(key_begin + key) * D) + ch);
        vv4 = __ldcg(reinterpret_cast<const uint4*>(vbase + (size_t)(key_begin + key) * D) + ch);
      }
      *reinterpret_cast<uint4*>(k_s + key * kStride + ch * 8) = kv4;
      *reinterpret_cast<uint4*>(v_s + key * kStride + ch * 8) = vv4;
    }
    asm volatile("cp.async.wait_all;\n" ::: "memory");
    cbar();
    // (c) one warp per 16 query rows
    const int row_tiles = (R + 15) / 16;
    if (warp < row_tiles) {
      uint32_t anc[2];   // the block has at most 8 rows here: the ancestor mask fits 32 bits
      uint32_t qf[kDSteps][4];
#pragma unroll
      for (int h = 0; h < 2; ++h) {
        const int r = warp * 16 + g + 8 * h;
        const bool ok = r < R;
        anc[h] = ok ? (uint32_t)p.bi.anc[b * p.T_max + r / G] : 0u;
        const __nv_bfloat16* qrow = q_s + (ok ? r : 0) * kStride;
#pragma unroll
        for (int kd = 0; kd < kDSteps; ++kd) {
          qf[kd][h] = ok ? *reinterpret_cast<const uint32_t*>(qrow + kd * 16 + 2 * t) : 0u;
          qf[kd][h + 2] = ok ? *reinterpret_cast<const uint32_t*>(qrow + kd * 16 + 8 + 2 * t) : 0u;
        }
      }
      const float scale_log2 = kLog2e / sqrtf((float)D);
      float s[kKeyTile / 8][4];
#pragma unroll
      for (int j = 0; j < kKeyTile / 8; ++j) {
        s[j][0] = s[j][1] = s[j][2] = s[j][3] = 0.f;
#pragma unroll
        for (int kd = 0; kd < kDSteps; ++kd) {
          const __nv_bfloat16* kr = k_s + (8 * j + g) * kStride + kd * 16 + 2 * t;
          mma16816_bf16(s[j], qf[kd][0], qf[kd][1], qf[kd][2], qf[kd][3], *reinterpret_cast<const uint32_t*>(kr),
                        *reinterpret_cast<const uint32_t*>(kr + 8));
        }
      }
      float row_max[2] = {-INFINITY, -INFINITY}, row_sum[2] = {0.f, 0.f};
#pragma unroll
      for (int j = 0; j < kKeyTile / 8; ++j) {
#pragma unroll
        for (int e = 0; e < 4; ++e) {
          const int h = e >> 1;
          const int key = key_begin + 8 * j + 2 * t + (e & 1);
          bool ok = key < key_end;
          if (ok && key >= P) ok = (anc[h] >> (key - P)) & 1u;
          const float v = ok ? s[j][e] * scale_log2 : -INFINITY;
          s[j][e] = v;
          row_max[h] = fmaxf(row_max[h], v);
        }
      }
      float m_use[2];
#pragma unroll
      for (int h = 0; h < 2; ++h) {
        row_max[h] = fmaxf(row_max[h], __shfl_xor_sync(0xffffffffu, row_max[h], 1));
        row_max[h] = fmaxf(row_max[h], __shfl_xor_sync(0xffffffffu, row_max[h], 2));
        m_use[h] = (row_max[h] == -INFINITY) ? 0.f : row_max[h];
      }
#pragma unroll
      for (int j = 0; j < kKeyTile / 8; ++j) {
#pragma unroll
        for (int e = 0; e < 4; ++e) {
          const float pr = exp2f(s[j][e] - m_use[e >> 1]);
          s[j][e] = pr;
          row_sum[e >> 1] += pr;
        }
      }
#pragma unroll
      for (int h = 0; h < 2; ++h) {
        row_sum[h] += __shfl_xor_sync(0xffffffffu, row_sum[h], 1);
        row_sum[h] += __shfl_xor_sync(0xffffffffu, row_sum[h], 2);
      }
      // O = P V in two halves of the head dimension (keeps the accumulators within the register budget)
#pragma unroll 1
      for (int half = 0; half < 2; ++half) {
        float o[D / 16][4];
#pragma unroll
        for (int i = 0; i < D / 16; ++i) o[i][0] = o[i][1] = o[i][2] = o[i][3] = 0.f;
#pragma unroll
        for (int kk = 0; kk < kKeyTile / 16; ++kk) {
          uint32_t ah[4], al[4];
          split_bf16(s[2 * kk][0], s[2 * kk][1], ah[0], al[0]);
          split_bf16(s[2 * kk][2], s[2 * kk][3], ah[1], al[1]);
          split_bf16(s[2 * kk + 1][0], s[2 * kk + 1][1], ah[2], al[2]);
          split_bf16(s[2 * kk + 1][2], s[2 * kk + 1][3], ah[3], al[3]);
#pragma unroll
          for (int dt = 0; dt < D / 32; ++dt) {
            uint32_t b0, b1, b2, b3;
            const int mat = lane >> 3, r = lane & 7;
            ldmatrix_x4_trans(b0, b1, b2, b3, v_s + (kk * 16 + (mat & 1) * 8 + r) * kStride + half * (D / 2) +
                                                  dt * 16 + (mat >> 1) * 8);
            mma16816_bf16(o[2 * dt], ah[0], ah[1], ah[2], ah[3], b0, b1);
            mma16816_bf16(o[2 * dt], al[0], al[1], al[2], al[3], b0, b1);
            mma16816_bf16(o[2 * dt + 1], ah[0], ah[1], ah[2], ah[3], b2, b3);
            mma16816_bf16(o[2 * dt + 1], al[0], al[1], al[2], al[3], b2, b3);
          }
        }
#pragma unroll
        for (int h = 0; h < 2; ++h) {
          const int r = warp * 16 + g + 8 * h;
          if (r >= p.attn_rpad) continue;
          float* op = o_s + r * D + half * (D / 2);
#pragma unroll
          for (int i = 0; i < D / 16; ++i)
            *reinterpret_cast<float2*>(op + 8 * i + 2 * t) = make_float2(o[i][2 * h], o[i][2 * h + 1]);
        }
      }
      if (t == 0) {
#pragma unroll
        for (int h = 0; h < 2; ++h) {
          const int r = warp * 16 + g + 8 * h;
          if (r >= p.attn_rpad) continue;
          ml_s[r * 2] = row_max[h];
          ml_s[r * 2 + 1] = row_sum[h];
        }
      }
    }

    // (d) The partial (un-normalised output, row maxima and sums) leaves as two bulk stores.  Then the
    //     CTAs of this (sequence, kv head) wait for one another (a bounded wait on the head's arrival
    //     count: all of them are resident) and share the merge: the CTA of chunk c takes the query rows
    //     c, c + nch, ...  A row's chunks are added in a fixed order whoever does it.
    const int nch = (Lk + kKeyTile - 1) / kKeyTile;
    const size_t slot0 = ((size_t)b * p.Hkv + hk) * p.attn_nchunk * p.attn_rpad;
    unsigned* arrivals = p.attn_count + (size_t)layer * p.B * p.Hkv + b * p.Hkv + hk;
    cbar();   // o_s and ml_s are complete
    if (threadIdx.x == 0) {
      const size_t slot = slot0 + (size_t)c * p.attn_rpad;
      asm volatile("fence.proxy.async.shared::cta;\n" ::: "memory");
      bulk_store(p.o_part + slot * D, o_s, (uint32_t)p.attn_rpad * D * 4);
      bulk_store(p.ml_part + slot * 2, ml_s, (uint32_t)p.attn_rpad * 8);
      asm volatile("cp.async.bulk.commit_group;\ncp.async.bulk.wait_group 0;\n" ::: "memory");
      __threadfence();   // this CTA's partial is visible before its arrival is
      atomicAdd(arrivals, 1u);
      int ok_flag = 1;
      if (c < R) {   // this CTA has rows to merge: wait for the other chunks
        const unsigned long long t0 = now_ns();
        unsigned polls = 0;
        while (true) {
          unsigned v;
          asm volatile("ld.acquire.gpu.global.u32 %0, [%1];\n" : "=r"(v) : "l"(arrivals) : "memory");
          if (v >= (unsigned)nch) break;
          if ((++polls & 63u) == 0 && (*abort_flag || now_ns() - t0 > wait_budget(abort_flag))) {
            atomicMin(p.status, QUASAR_ERR_TIMEOUT);
            *abort_flag = 1;
            ok_flag = 0;
            break;
          }
        }
      }
      *last_flag = ok_flag;
    }
    cbar();
    if (*last_flag) {
      // Two rows at a time, half of the warps each: warp ws of a half adds the chunks ws, ws + NW/2, ...
      // of its row (lane l: four output dimensions); the warps' sums meet in shared memory in warp order.
      // All loads of a row - every chunk's (m, l) for the row maximum, this warp's chunks' partial
      // outputs - are issued before the first of them is used: one round trip to L2 per pair of rows.
      float* part = o_s;                                   // [NW][D + 4] floats; the partial has left
      constexpr int kPS = 128 + 4;
      constexpr int kHalf = NW / 2, kPre = 4;
      const int half = warp / kHalf, ws = warp % kHalf;
#pragma unroll 1
      for (int r0 = c; r0 < R; r0 += 2 * nch) {
        const int r = r0 + half * nch;
        const bool live = r < R;
        float acc[4] = {0.f, 0.f, 0.f, 0.f};
        float den = 0.f;
        if (live) {
          float2 ml[kPre];
          float4 ov[kPre];
#pragma unroll
          for (int q = 0; q < kPre; ++q) {
            const int cc = ws + q * kHalf;
            ml[q] = make_float2(-INFINITY, 0.f);
            ov[q] = make_float4(0.f, 0.f, 0.f, 0.f);
            if (cc < nch) {
              const size_t sidx = slot0 + (size_t)cc * p.attn_rpad + r;
              ml[q] = __ldcg(reinterpret_cast<const float2*>(p.ml_part + sidx * 2));
              if constexpr (D == 128) {
                ov[q] = __ldcg(reinterpret_cast<const float4*>(p.o_part + sidx * D) + lane);
              } else {
                const float2 o2 = __ldcg(reinterpret_cast<const float2*>(p.o_part + sidx * D) + lane);
                ov[q] = make_float4(o2.x, o2.y, 0.f, 0.f);
              }
            }
          }
          float mx = -INFINITY;
          for (int cc = lane; cc < nch; cc += 32) mx = fmaxf(mx, __ldcg(p.ml_part + (slot0 + (size_t)cc * p.attn_rpad + r) * 2));
#pragma unroll
          for (int o = 16; o > 0; o >>= 1) mx = fmaxf(mx, __shfl_xor_sync(0xffffffffu, mx, o));
#pragma unroll
          for (int q = 0; q < kPre; ++q) {   // chunks in ascending order, as below
            const float w = ml[q].x == -INFINITY ? 0.f : exp2f(ml[q].x - mx);
            den += w * ml[q].y;
            acc[0] += w * ov[q].x; acc[1] += w * ov[q].y; acc[2] += w * ov[q].z; acc[3] += w * ov[q].w;
          }
#pragma unroll 1
          for (int cc = ws + kPre * kHalf; cc < nch; cc += kHalf) {   // long sequences: the chunks beyond the first kPre per warp
            const size_t sidx = slot0 + (size_t)cc * p.attn_rpad + r;
            const float2 m2 = __ldcg(reinterpret_cast<const float2*>(p.ml_part + sidx * 2));
            const float w = m2.x == -INFINITY ? 0.f : exp2f(m2.x - mx);
            den += w * m2.y;
            if constexpr (D == 128) {
              const float4 o4 = __ldcg(reinterpret_cast<const float4*>(p.o_part + sidx * D) + lane);
              acc[0] += w * o4.x; acc[1] += w * o4.y; acc[2] += w * o4.z; acc[3] += w * o4.w;
            } else {
              const float2 o2 = __ldcg(reinterpret_cast<const float2*>(p.o_part + sidx * D) + lane);
              acc[0] += w * o2.x; acc[1] += w * o2.y;
            }
          }
        }
        cbar();   // the previous rows' sums have been read
        *reinterpret_cast<float4*>(part + warp * kPS + lane * 4) = make_float4(acc[0], acc[1], acc[2], acc[3]);
        if (lane == 0) part[warp * kPS + 128] = den;
        cbar();
        if (ws == 0 && live) {
          float tot[4] = {0.f, 0.f, 0.f, 0.f};
          float dsum = 0.f;
#pragma unroll
          for (int w = 0; w < kHalf; ++w) {
            const float4 v = *reinterpret_cast<const float4*>(part + (half * kHalf + w) * kPS + lane * 4);
            tot[0] += v.x; tot[1] += v.y; tot[2] += v.z; tot[3] += v.w;
            dsum += part[(half * kHalf + w) * kPS + 128];
          }
          const float inv = 1.0f / dsum;
          const int i = r / G, hq = hk * G + (r % G);
          const int m = b * p.T_max + i;
          const size_t off = (size_t)m * p.Hq * D + (size_t)hq * D + lane * (D / 32);
          __nv_bfloat16* dst = p.attn + off;
          float amax = 0.f;
#pragma unroll
          for (int e = 0; e < D / 64; ++e) {
            const __nv_bfloat162 pr = __floats2bfloat162_rn(tot[2 * e] * inv, tot[2 * e + 1] * inv);
            reinterpret_cast<__nv_bfloat162*>(dst)[e] = pr;
            const float2 back = __bfloat1622float2(pr);
            if (want_amax) reinterpret_cast<__half2*>(p.attn16 + off)[e] = __floats2half2_rn(back.x, back.y);
            amax = fmaxf(amax, fmaxf(fabsf(back.x), fabsf(back.y)));
          }
          if (want_amax) {   // row maximum of the o projection's operand
#pragma unroll
            for (int o = 16; o > 0; o >>= 1) amax = fmaxf(amax, __shfl_xor_sync(0xffffffffu, amax, o));
            if (lane == 0 && amax > 0.f) atomicMax(p.amax_buf + (4 * layer + 1) * 8 + m, __float_as_uint(amax));
          }
        }
      }
    }
  }
  asm volatile("cp.async.wait_all;\n" ::: "memory");   // a prefetch whose item was skipped has landed before the tiles are reused
}

// final phase on CTA 0: arg-max over the per-CTA candidates, then greedy acceptance
__device__ void accept_phase(const MegaParams& p, int ncta) {
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  for (int m = warp; m < p.M; m += NW) {
    float best = -INFINITY;
    int bi = 0x7fffffff;
    for (int c = lane; c < ncta; c += 32) {
      const float v = __ldcg(p.cand_val + (size_t)c * 8 + m);
      const int i = __ldcg(p.cand_idx + (size_t)c * 8 + m);
      if (v > best || (v == best && i < bi)) { best = v; bi = i; }
    }
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) {
      const float ob = __shfl_xor_sync(0xffffffffu, best, o);
      const int oi = __shfl_xor_sync(0xffffffffu, bi, o);
      if (ob > best || (ob == best && oi < bi)) { best = ob; bi = oi; }
    }
    if (lane == 0) p.top1[m] = bi == 0x7fffffff ? 0 : bi;
  }
  cbar();
  if ((int)threadIdx.x < p.B) {
    const int b = threadIdx.x, base = b * p.T_max;
    if (!p.bi.valid[b]) {   // a skipped sequence: -1 tells quasar_kv_commit to leave its cache and seq_len alone
      p.accept_len[b] = -1;
      p.bonus[b] = -1;
      if (p.accept_path) for (int d = 0; d < p.T_max; ++d) p.accept_path[base + d] = -1;
    } else {
      const int T = p.block_len[b];
      int cur = 0, n = 0;
      if (p.accept_path) p.accept_path[base] = 0;
      while (true) {
        int nxt = -1;
        const int want = p.top1[base + cur];
        for (int c = cur + 1; c < T; ++c) {
          const int par = p.parents ? p.parents[base + c] : c - 1;
          if (par == cur && p.tokens[base + c] == want) { nxt = c; break; }
        }
        if (nxt < 0) break;
        cur = nxt;
        ++n;
        if (p.accept_path) p.accept_path[base + n] = cur;
      }
      p.accept_len[b] = n;
      p.bonus[b] = p.top1[base + cur];
      if (p.accept_path) for (int d = n + 1; d < p.T_max; ++d) p.accept_path[base + d] = -1;
    }
  }
}

template <bool W_INT8, int D>
__global__ void __launch_bounds__(kThreads, 1) verify_megakernel(const MegaParams p) {
  extern __shared__ __align__(128) unsigned char smem[];
  const int cta = blockIdx.x, ncta = gridDim.x;
  const int warp = threadIdx.x >> 5;
  float* red = reinterpret_cast<float*>(smem + kRingBytes);
  unsigned char* x_s = smem + kRingBytes + kRedBytes;   // operand staging; the attention tiles live in the same bytes
  __nv_bfloat16* k_s = reinterpret_cast<__nv_bfloat16*>(x_s);
  __nv_bfloat16* v_s = reinterpret_cast<__nv_bfloat16*>(x_s + kKvTileBytes);
  __nv_bfloat16* q_s = reinterpret_cast<__nv_bfloat16*>(x_s + 2 * kKvTileBytes);
  float* misc = reinterpret_cast<float*>(x_s + kStageBufBytes);
  volatile int* abort_flag = reinterpret_cast<volatile int*>(misc + kMiscAbort);
  uint64_t* bars = reinterpret_cast<uint64_t*>(reinterpret_cast<unsigned char*>(misc) + kMiscBarBytes);
  Pipe pipe{smem, bars, bars + kStages, abort_flag, p.status};
  uint64_t* xbar = bars + 2 * kStages;   // the operand's bulk copies have landed (xbar[1]: second buffer of the attention merge)

  if (threadIdx.x == 0) {
    *abort_flag = 0;
    *reinterpret_cast<volatile unsigned long long*>(abort_flag + 2) = p.wait_budget_ns;
    for (int s = 0; s < kStages; ++s) {
      mbar_init(pipe.full + s, 1);     // the producer's arrive.expect_tx; the bytes complete the phase
      mbar_init(pipe.empty + s, NW);   // one arrival per consumer warp
    }
    mbar_init(xbar, 1);
    mbar_init(xbar + 1, 1);
    asm volatile("fence.mbarrier_init.release.cluster;\n" ::: "memory");
  }
  if (threadIdx.x == 32) reinterpret_cast<MegaJob*>(misc + kMiscJob)[0] = p.jobs[0];
  if (threadIdx.x < 8) {  // running arg-max of this CTA
    misc[kMiscRunV + threadIdx.x] = -INFINITY;
    reinterpret_cast<int*>(misc + kMiscRunI)[threadIdx.x] = 0x7fffffff;
  }
  __syncthreads();

  if (warp == NW) {  // the weight stream
    producer_loop<W_INT8>(p, pipe, cta, ncta);
    return;
  }

  int slot = 0;
  uint32_t phase = 0, xphase = 0, xphase2 = 0;
  // (barrier_extra is zero except in the test of the failure path: a barrier that expects more arrivals than
  // there are thread blocks cannot complete, so its first wait runs into the budget)
  GridSync gs{p.barrier, p.status, (unsigned)ncta + p.barrier_extra, 0u, abort_flag};
  bool ok = true;
  prep_phase(p, misc, cta, ncta);
  gs.arrive();
  // the GEMMs of the pass in order (qkv, o, gate+up, down per layer, then the LM head); attention follows every qkv
  for (int job = 0; job < p.n_jobs && ok; ++job) {
    // (every GEMM phase waits, inside, for the grid barrier that the phase before it arrived at)
    if (!(ok = GemmPhase<W_INT8>::run(p, job, pipe, slot, phase, red, misc, x_s, xbar, xphase, cta, ncta, gs))) break;
    if (job == p.n_jobs - 1) break;   // the LM head is followed by the candidate exchange below
    gs.arrive();
    if ((job & 3) == 0) {
      attention_prefetch<D>(p, job >> 2, k_s, v_s, cta);   // reads the cached prefix only: nothing of this phase
      if (!(ok = gs.wait())) break;
      attention_phase<D>(p, job >> 2, W_INT8, k_s, v_s, q_s, misc, xbar, xphase, xphase2, cta, ncta);
      gs.arrive();
    }
  }
  if (ok) {
    cbar();
    if (threadIdx.x < 8) {
      p.cand_val[(size_t)cta * 8 + threadIdx.x] = misc[kMiscRunV + threadIdx.x];
      p.cand_idx[(size_t)cta * 8 + threadIdx.x] = reinterpret_cast<int*>(misc + kMiscRunI)[threadIdx.x];
    }
    ok = gs.sync();
    if (ok && cta == 0) accept_phase(p, ncta);
  }
  if (!ok && threadIdx.x == 0) {
    *abort_flag = 1;  // tells the producer to stop issuing
    // an operand chunk may have been requested and never waited for: let it land (it takes a few
    // microseconds at most) before the CTA gives its shared memory back
    const unsigned long long t0 = now_ns();
    while (!mbar_try(xbar, xphase) && now_ns() - t0 < 100000ull) {}
  }
}

// ---- model creation: permute every CTA's row range into its consumption order ------------------
// One thread block per (tile, CTA).  The destination has the size of the source and every CTA's
// range starts where its rows start in the source; inside the range the blocks follow the
// schedule above.  int8 weights get their sign bits flipped (see u8x4_to_f16x4).
template <bool W_INT8>
__global__ void __launch_bounds__(256) repack_kernel(const unsigned char* __restrict__ w, unsigned char* __restrict__ wp,
                                                     int N, int K, int kind, int ncta) {
  constexpr int kElemBytes = W_INT8 ? 1 : 2;
  const int cta = blockIdx.y, tile_g = blockIdx.x;
  JobView v;
  job_split(kind, N, K, cta, ncta, v);
  const int kChunkBytes = v.chunk * kElemBytes;
  if (tile_g >= v.tiles) return;
  const int mult = kind == kJobGateUp ? 2 : 1;
  const int tg = tile_g / GT, tile = tile_g % GT;
  const int gt = min(GT, v.tiles - tg * GT);
  int rows_in_group = 0;
  for (int i = 0; i < gt; ++i) rows_in_group += tile_rows(v, tg * GT + i);
  const size_t rows_before_group = (size_t)mult * tg * GT * v.rows_per_tile;   // every earlier tile is full
  const size_t rows_before_in_group = (size_t)mult * tile * v.rows_per_tile;
  const int nr = tile_rows(v, tile_g);
  const size_t kbytes = (size_t)K * kElemBytes;
  unsigned char* region = wp + (size_t)mult * v.u0 * kbytes;
  for (int kc = 0; kc < v.nchunks; ++kc) {
    const int cb = (int)min((size_t)kChunkBytes, kbytes - (size_t)kc * kChunkBytes);
    const size_t chunk_off = rows_before_group * kbytes + (size_t)rows_in_group * kc * kChunkBytes + rows_before_in_group * cb;
    for (int b0 = 0; b0 < cb; b0 += kRowBytes) {
      const int pb = min(kRowBytes, cb - b0);
      unsigned char* blk = region + chunk_off + (size_t)nr * b0;
      const int per_row = pb / 16;
      for (int idx = threadIdx.x; idx < nr * per_row; idx += blockDim.x) {
        const int row = idx / per_row, ch = idx % per_row;
        const int n = block_row_to_global(v, tile_g, row);
        uint4 val = __ldg(reinterpret_cast<const uint4*>(w + (size_t)n * kbytes + (size_t)kc * kChunkBytes + b0) + ch);
        if (W_INT8) { val.x ^= 0x80808080u; val.y ^= 0x80808080u; val.z ^= 0x80808080u; val.w ^= 0x80808080u; }
        const int dch = (pb & 127) == 0 ? ch ^ ((row & 1) << 2) : ch;
        *reinterpret_cast<uint4*>(blk + (size_t)row * pb + dch * 16) = val;
      }
    }
  }
}

template <bool W_INT8, int D>
int launch_variant(const MegaParams& p, int ncta, cudaStream_t stream) {
  static bool configured = false;
  auto kernel = verify_megakernel<W_INT8, D>;
  if (!configured) {
    QUASAR_CUDA_CHECK(cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, kSmemBytes));
    configured = true;
  }
  void* args[] = {const_cast<MegaParams*>(&p)};
  QUASAR_CUDA_CHECK(cudaLaunchCooperativeKernel(reinterpret_cast<void*>(kernel), dim3(ncta), dim3(kThreads), args,
                                                (size_t)kSmemBytes, stream));
  count_launch();
  return QUASAR_OK;
}

}  // namespace


int launch_repack(const void* w, void* wp, int N, int K, int kind, int weight_dtype, int ncta, cudaStream_t stream) {
  const int units = kind == kJobGateUp ? N / 2 : N;
  const int rpt = kind == kJobGateUp ? 8 : 16;
  const int max_units = (units + ncta - 1) / ncta;
  dim3 grid((max_units + rpt - 1) / rpt, ncta);
  if (weight_dtype == QUASAR_W_INT8)
    repack_kernel<true><<<grid, 256, 0, stream>>>(reinterpret_cast<const unsigned char*>(w),
                                                  reinterpret_cast<unsigned char*>(wp), N, K, kind, ncta);
  else
    repack_kernel<false><<<grid, 256, 0, stream>>>(reinterpret_cast<const unsigned char*>(w),
                                                   reinterpret_cast<unsigned char*>(wp), N, K, kind, ncta);
  QUASAR_LAUNCH_CHECK();
  return QUASAR_OK;
}

bool mega_supported(int M, int T_max, int Hq, int Hkv, int D) {
  return M <= 8 && (Hq / Hkv) * T_max <= kMaxRowsAttn && (D == 64 || D == 128);
}

int mega_attn_nchunk(int s_max) { return (s_max + kKeyTile - 1) / kKeyTile; }
int mega_attn_rpad(int T_max, int Hq, int Hkv) { return ((Hq / Hkv) * T_max + 15) / 16 * 16; }

int mega_grid_size(int weight_dtype, int D, int* ncta_out) {
  int dev = 0, sms = 0, per_sm = 0;
  QUASAR_CUDA_CHECK(cudaGetDevice(&dev));
  QUASAR_CUDA_CHECK(cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev));
  const void* k = nullptr;
  if (weight_dtype == QUASAR_W_INT8) k = D == 128 ? (const void*)verify_megakernel<true, 128> : (const void*)verify_megakernel<true, 64>;
  else k = D == 128 ? (const void*)verify_megakernel<false, 128> : (const void*)verify_megakernel<false, 64>;
  QUASAR_CUDA_CHECK(cudaFuncSetAttribute(k, cudaFuncAttributeMaxDynamicSharedMemorySize, kSmemBytes));
  QUASAR_CUDA_CHECK(cudaOccupancyMaxActiveBlocksPerMultiprocessor(&per_sm, k, kThreads, (size_t)kSmemBytes));
  if (per_sm < 1) {
    set_error("persistent kernel does not fit on an SM (%d bytes of shared memory)", kSmemBytes);
    return QUASAR_ERR_CUDA;
  }
  if (sms < 8) {
    set_error("persistent kernel needs at least 8 SMs");
    return QUASAR_ERR_CUDA;
  }
  *ncta_out = sms;
  return QUASAR_OK;
}

int launch_verify_mega(const MegaParams& p, int weight_dtype, int D, int ncta, cudaStream_t stream) {
  if (weight_dtype == QUASAR_W_INT8) {
    return D == 128 ? launch_variant<true, 128>(p, ncta, stream) : launch_variant<true, 64>(p, ncta, stream);
  }
  return D == 128 ? launch_variant<false, 128>(p, ncta, stream) : launch_variant<false, 64>(p, ncta, stream);
}

}  // namespace quasar
