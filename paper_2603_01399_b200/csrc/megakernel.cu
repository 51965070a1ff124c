// The whole verification pass (Section 3.1 "Verification", Section 3.3) as ONE persistent
// cooperative kernel: one CTA per SM, every step of the pass a phase separated by a grid
// barrier.  Section 3.4 models the pass as  T ~= M * bytes / BW : the pass is one long read
// of the weights, so the design goal is that this read never stops.
//
//  * Every warp owns a private ring of shared-memory stages that it fills with cp.async
//    from a STATIC schedule covering all GEMMs of the pass.  The schedule does not depend on
//    activations, so a warp keeps prefetching the next GEMM's weights while the CTA is in
//    an epilogue, an attention phase or a grid barrier (160 KB in flight per SM).
//  * Each weight matrix is cut into contiguous row ranges, one per CTA, balanced to a single
//    row, so all SMs stream the same number of bytes and no cross-CTA reduction exists.
//    Inside a CTA the 16 warps split the contraction index; their partial sums meet in
//    shared memory in a fixed order (deterministic results).
//  * int8 -> bf16 in registers, mma.m16n8k16 with the weights as the 16-row operand and the
//    <= 8 activation rows as the 8-wide operand held in registers for a whole phase.
//  * RMSNorm is fused into the operand load of the following GEMM, SwiGLU / residual adds
//    into the GEMM epilogues, QK-RMSNorm + RoPE + KV append into the attention phase.
//
// Every wait is bounded: a grid barrier that does not complete within its poll budget sets
// QUASAR_ERR_TIMEOUT in the status word and the CTA leaves (after draining its copies).
#include <cooperative_groups.h>
#include <math.h>

#include "common.cuh"
#include "megakernel.cuh"

namespace quasar {

namespace {

constexpr int NW = kMegaWarps;          // warps per CTA
constexpr int kThreads = NW * 32;
constexpr int kStageBytes = 2048;       // 16 weight rows x 128 bytes
constexpr int kChunk = 4096;            // contraction elements the CTA covers per chunk
constexpr int kSlice = kChunk / NW;     // contraction elements one warp covers per chunk
constexpr int kStages = 80 / NW;        // ring depth per warp (160 KB of stages per CTA)
constexpr int kXr = kSlice / 32;        // 16-byte registers holding this thread's share of the operand slice
constexpr int GT = 4;                   // 16-row tiles accumulated together before a reduction
constexpr int kKeyTile = 64;
constexpr int kMaxRowsAttn = 64;        // query rows (heads-in-group x block rows) per kv head
constexpr float kLog2e = 1.4426950408889634f;
constexpr unsigned kBarrierPolls = 4u << 20;

// ---- shared memory map --------------------------------------------------------------------
constexpr int kRingBytes = NW * kStages * kStageBytes;                   // 163840
constexpr int kRedBytes = NW * GT * 128 * 4;                             // 32768
constexpr int kKvTileBytes = kKeyTile * (128 + 8) * 2;                   // 17408 (D = 128)
constexpr int kUnionBytes = (2 * kKvTileBytes > kRedBytes) ? 2 * kKvTileBytes : kRedBytes;
constexpr int kQTileBytes = kMaxRowsAttn * (128 + 8) * 2;                // 17408
constexpr int kMiscBytes = 2048;
constexpr int kSmemBytes = kRingBytes + kUnionBytes + kQTileBytes + kMiscBytes;

__device__ __forceinline__ void cp_async16(void* smem, const void* gmem, bool valid) {
  const uint32_t d = (uint32_t)__cvta_generic_to_shared(smem);
  const int n = valid ? 16 : 0;
  asm volatile("cp.async.cg.shared.global [%0], [%1], 16, %2;\n" ::"r"(d), "l"(gmem), "r"(n) : "memory");
}
__device__ __forceinline__ void cp_async_commit() { asm volatile("cp.async.commit_group;\n" ::: "memory"); }
template <int N>
__device__ __forceinline__ void cp_async_wait() { asm volatile("cp.async.wait_group %0;\n" ::"n"(N) : "memory"); }

__device__ __forceinline__ void mma16816(float (&c)[4], uint32_t a0, uint32_t a1, uint32_t a2, uint32_t a3,
                                         uint32_t b0, uint32_t b1) {
  asm volatile(
      "mma.sync.aligned.m16n8k16.row.col.f32.bf16.bf16.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%0,%1,%2,%3};\n"
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

// Four signed bytes -> four bf16 (exact), see the skinny GEMM.
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

// ---- the static weight schedule -----------------------------------------------------------
// Position of one warp in the sequence of ring stages of the whole pass.  Order:
// job -> tile group -> contraction chunk -> tile in group -> 128-byte piece of the warp's slice.
struct JobView {
  const unsigned char* w;
  int K, units, u0, u1, rows_per_tile, tiles, ngroups, nchunks, kind, n_rows;
};

__device__ __forceinline__ JobView job_view(const MegaJob* jobs, int j, int cta, int ncta) {
  JobView v;
  const MegaJob jb = jobs[j];
  v.w = reinterpret_cast<const unsigned char*>(jb.w);
  v.K = jb.K;
  v.kind = jb.kind;
  v.n_rows = jb.N;
  v.units = (jb.kind == kJobGateUp) ? jb.N / 2 : jb.N;
  v.u0 = (int)(((long long)cta * v.units) / ncta);
  v.u1 = (int)(((long long)(cta + 1) * v.units) / ncta);
  v.rows_per_tile = (jb.kind == kJobGateUp) ? 8 : 16;
  v.tiles = (v.u1 - v.u0 + v.rows_per_tile - 1) / v.rows_per_tile;
  v.ngroups = (v.tiles + GT - 1) / GT;
  v.nchunks = (jb.K + kChunk - 1) / kChunk;
  return v;
}

// global weight row behind ring row r (0..15) of tile `tile`, or -1 when the slot is padding
__device__ __forceinline__ int ring_row_to_global(const JobView& v, int tile, int r) {
  if (v.kind == kJobGateUp) {
    const int p = v.u0 + tile * 8 + (r & 7);
    if (p >= v.u1) return -1;
    return (r < 8) ? p : v.units + p;
  }
  const int n = v.u0 + tile * 16 + r;
  return n < v.u1 ? n : -1;
}

template <bool W_INT8>
struct Producer {
  static constexpr int kStageElems = W_INT8 ? 128 : 64;
  static constexpr int KB = kSlice / kStageElems;    // ring stages per (tile, chunk) per warp
  const MegaJob* jobs;
  int n_jobs, cta, ncta, warp, lane;
  int job, tg, kc, tile, kb;
  JobView v;
  bool done;

  __device__ void init(const MegaJob* j, int nj, int c, int nc, int w, int l) {
    jobs = j; n_jobs = nj; cta = c; ncta = nc; warp = w; lane = l;
    job = -1; tg = kc = tile = kb = 0; done = false;
    next_job();
  }
  __device__ void next_job() {
    while (true) {
      ++job;
      if (job >= n_jobs) { done = true; return; }
      v = job_view(jobs, job, cta, ncta);
      if (v.tiles > 0) break;
    }
    tg = kc = tile = kb = 0;
  }
  __device__ void advance() {
    if (++kb < KB) return;
    kb = 0;
    const int gt = min(GT, v.tiles - tg * GT);
    if (++tile < gt) return;
    tile = 0;
    if (++kc < v.nchunks) return;
    kc = 0;
    if (++tg < v.ngroups) return;
    next_job();
  }
  // issue the copies of the current stage into `slot` and move on (always exactly one commit group)
  __device__ void fetch(unsigned char* slot) {
    if (!done) {
      const int kbase = kc * kChunk + warp * kSlice + kb * kStageElems;
      const int t_global = tg * GT + tile;
      constexpr int kElemsPer16 = W_INT8 ? 16 : 8;
#pragma unroll
      for (int i = 0; i < 4; ++i) {
        const int q = lane + 32 * i;
        const int r = q >> 3, c = q & 7;
        const int n = ring_row_to_global(v, t_global, r);
        const int k = kbase + c * kElemsPer16;
        const bool ok = (n >= 0) && (k < v.K);
        const unsigned char* src = v.w + ((size_t)(ok ? n : 0) * v.K + (ok ? k : 0)) * (W_INT8 ? 1 : 2);
        cp_async16(slot + r * 128 + ((c * 16) ^ ((r & 1) << 6)), src, ok);
      }
      advance();
    }
    cp_async_commit();
  }
};

// ---- bounded grid barrier -----------------------------------------------------------------
struct GridSync {
  unsigned* counter;
  int32_t* status;
  unsigned ncta;
  unsigned epoch;
  int* abort_flag;  // shared memory
  __device__ bool sync() {
    __syncthreads();
    if (threadIdx.x == 0) {
      ++epoch;
      __threadfence();
      atomicAdd(counter, 1u);
      const unsigned target = epoch * ncta;
      unsigned polls = 0;
      while (true) {
        unsigned v;
        asm volatile("ld.acquire.gpu.global.u32 %0, [%1];\n" : "=r"(v) : "l"(counter) : "memory");
        if (v >= target) break;
        if (++polls > kBarrierPolls) {
          atomicMin(status, QUASAR_ERR_TIMEOUT);
          *abort_flag = 1;
          break;
        }
        __nanosleep(20);
      }
    } else {
      epoch++;
    }
    __syncthreads();
    return *abort_flag == 0;
  }
};

// ---- operand load: the <= 8 activation rows of this warp's contraction slice ------------------
// xr[0..kXr): for int8 weights step s (64 elements) uses xr[2s], xr[2s+1] (16 bf16 of row g at
// k = base + s*64 + t*16); for bf16 weights step s (32 elements) uses xr[s] (8 bf16 at base + s*32 + t*8).
template <bool W_INT8>
__device__ __forceinline__ void load_x_raw(uint4 (&xr)[kXr], const __nv_bfloat16* src, int ld, int M, int K, int kbase,
                                           int g, int t) {
#pragma unroll
  for (int i = 0; i < kXr; ++i) {
    const int k = W_INT8 ? (kbase + (i >> 1) * 64 + t * 16 + (i & 1) * 8) : (kbase + i * 32 + t * 8);
    xr[i] = make_uint4(0, 0, 0, 0);
    if (g < M && k < K) xr[i] = __ldcg(reinterpret_cast<const uint4*>(src + (size_t)g * ld + k));
  }
}

template <bool W_INT8>
__device__ __forceinline__ void apply_norm(uint4 (&xr)[kXr], const __nv_bfloat16* gain, float r, int K, int kbase,
                                           int t) {
#pragma unroll
  for (int i = 0; i < kXr; ++i) {
    const int k = W_INT8 ? (kbase + (i >> 1) * 64 + t * 16 + (i & 1) * 8) : (kbase + i * 32 + t * 8);
    if (k < K) {
      const uint4 gv = __ldg(reinterpret_cast<const uint4*>(gain + k));
      const __nv_bfloat162* xp = reinterpret_cast<const __nv_bfloat162*>(&xr[i]);
      const __nv_bfloat162* gp = reinterpret_cast<const __nv_bfloat162*>(&gv);
      uint32_t o[4];
#pragma unroll
      for (int e = 0; e < 4; ++e) {
        const float2 xf = __bfloat1622float2(xp[e]);
        const float2 gf = __bfloat1622float2(gp[e]);
        o[e] = pack_bf16(xf.x * r * gf.x, xf.y * r * gf.y);
      }
      xr[i] = make_uint4(o[0], o[1], o[2], o[3]);
    }
  }
}

__device__ __forceinline__ float sumsq(const uint4 (&xr)[kXr]) {
  float s = 0.f;
#pragma unroll
  for (int i = 0; i < kXr; ++i) {
    const __nv_bfloat162* xp = reinterpret_cast<const __nv_bfloat162*>(&xr[i]);
#pragma unroll
    for (int e = 0; e < 4; ++e) {
      const float2 f = __bfloat1622float2(xp[e]);
      s += f.x * f.x + f.y * f.y;
    }
  }
  return s;
}

template <bool W_INT8>
__device__ __forceinline__ void consume_stage(const unsigned char* stage, int kb, const uint4 (&xr)[kXr],
                                              float (&acc)[4], int g, int t) {
#pragma unroll
  for (int s = 0; s < 2; ++s) {
    const int off = (s * 64 + t * 16) ^ ((g & 1) << 6);
    const uint4 wa = *reinterpret_cast<const uint4*>(stage + g * 128 + off);
    const uint4 wb = *reinterpret_cast<const uint4*>(stage + (g + 8) * 128 + off);
    const int step = kb * 2 + s;
    if (W_INT8) {
      const uint4 x0 = xr[2 * step], x1 = xr[2 * step + 1];
      uint32_t a0, a1, a2, a3;
      s8x4_to_bf16x4(wa.x, a0, a2); s8x4_to_bf16x4(wb.x, a1, a3);
      mma16816(acc, a0, a1, a2, a3, x0.x, x0.y);
      s8x4_to_bf16x4(wa.y, a0, a2); s8x4_to_bf16x4(wb.y, a1, a3);
      mma16816(acc, a0, a1, a2, a3, x0.z, x0.w);
      s8x4_to_bf16x4(wa.z, a0, a2); s8x4_to_bf16x4(wb.z, a1, a3);
      mma16816(acc, a0, a1, a2, a3, x1.x, x1.y);
      s8x4_to_bf16x4(wa.w, a0, a2); s8x4_to_bf16x4(wb.w, a1, a3);
      mma16816(acc, a0, a1, a2, a3, x1.z, x1.w);
    } else {
      const uint4 x0 = xr[step];
      mma16816(acc, wa.x, wb.x, wa.y, wb.y, x0.x, x0.y);
      mma16816(acc, wa.z, wb.z, wa.w, wb.w, x0.z, x0.w);
    }
  }
}

// ---- one GEMM phase -----------------------------------------------------------------------
template <bool W_INT8>
struct GemmPhase {
  static constexpr int KB = Producer<W_INT8>::KB;

  __device__ __noinline__ static void run(const MegaParams& p, int job, Producer<W_INT8>& prod_io,
                                          unsigned char* ring, unsigned& cstage_io, float* red, float* misc, int cta,
                                          int ncta) {
    Producer<W_INT8> prod = prod_io;  // registers while the phase runs
    unsigned cstage = cstage_io;
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31, g = lane >> 2, t = lane & 3;
    const JobView v = job_view(p.jobs, job, cta, ncta);
    const MegaJob jb = p.jobs[job];
    const int M = p.M;
    const bool normed = jb.gain != nullptr;
    const __nv_bfloat16* xsrc = jb.kind == kJobO ? p.attn : (jb.kind == kJobDown ? p.act : p.x);
    const int ld = jb.K;

    // RMSNorm factor of every row (the operand of a normed GEMM is h = x * r * gain)
    float rnorm = 1.f;
    uint4 xr[kXr];
    bool have_x = false;
    if (normed) {
      float ss = 0.f;
      for (int kc = 0; kc < v.nchunks; ++kc) {
        load_x_raw<W_INT8>(xr, xsrc, ld, M, jb.K, kc * kChunk + warp * kSlice, g, t);
        ss += sumsq(xr);
      }
      ss += __shfl_xor_sync(0xffffffffu, ss, 1);
      ss += __shfl_xor_sync(0xffffffffu, ss, 2);
      if (t == 0) misc[warp * 8 + g] = ss;
      __syncthreads();
      float tot = 0.f;
#pragma unroll
      for (int w = 0; w < NW; ++w) tot += misc[w * 8 + g];
      rnorm = 1.0f / sqrtf(tot / (float)jb.K + p.rms_eps);
      __syncthreads();
      if (v.nchunks == 1) {
        apply_norm<W_INT8>(xr, jb.gain, rnorm, jb.K, warp * kSlice, t);
        have_x = true;
      }
    }

    // per-CTA arg-max state of the LM head (thread tid < 8*... handled in the epilogue)
    for (int tg = 0; tg < v.ngroups; ++tg) {
      const int gt = min(GT, v.tiles - tg * GT);
      float acc[GT][4];
#pragma unroll
      for (int i = 0; i < GT; ++i) acc[i][0] = acc[i][1] = acc[i][2] = acc[i][3] = 0.f;
      for (int kc = 0; kc < v.nchunks; ++kc) {
        if (!have_x) {
          load_x_raw<W_INT8>(xr, xsrc, ld, M, jb.K, kc * kChunk + warp * kSlice, g, t);
          if (normed) apply_norm<W_INT8>(xr, jb.gain, rnorm, jb.K, kc * kChunk + warp * kSlice, t);
          have_x = (v.nchunks == 1);
        }
#pragma unroll
        for (int tile = 0; tile < GT; ++tile) {
          if (tile < gt) {
#pragma unroll
            for (int kb = 0; kb < KB; ++kb) {
              cp_async_wait<kStages - 2>();
              __syncwarp();
              prod.fetch(ring + ((cstage + kStages - 1) % kStages) * kStageBytes);
              consume_stage<W_INT8>(ring + (cstage % kStages) * kStageBytes, kb, xr, acc[tile], g, t);
              ++cstage;
            }
          }
        }
      }
      // ---- cross-warp reduction in a fixed order, then the fused epilogue ----
#pragma unroll
      for (int tile = 0; tile < GT; ++tile) {
        float* r = red + ((warp * GT + tile) * 16) * 8;
        *reinterpret_cast<float2*>(r + g * 8 + 2 * t) = make_float2(acc[tile][0], acc[tile][1]);
        *reinterpret_cast<float2*>(r + (g + 8) * 8 + 2 * t) = make_float2(acc[tile][2], acc[tile][3]);
      }
      __syncthreads();
      epilogue(p, jb, v, tg, gt, red, misc);
      __syncthreads();
    }
    prod_io = prod;
    cstage_io = cstage;
  }

  __device__ static float reduce_at(const float* red, int tile, int row, int col) {
    float s = 0.f;
#pragma unroll
    for (int w = 0; w < NW; ++w) s += red[((w * GT + tile) * 16 + row) * 8 + col];
    return s;
  }

  __device__ static void epilogue(const MegaParams& p, const MegaJob& jb, const JobView& v, int tg, int gt,
                                  const float* red, float* misc) {
    const int M = p.M;
    if (jb.kind == kJobGateUp) {
      const int F = v.units;
      for (int e = threadIdx.x; e < gt * 8 * 8; e += kThreads) {
        const int r = e & 7, col = (e >> 3) & 7, tile = e >> 6;
        const int pair = v.u0 + (tg * GT + tile) * 8 + r;
        if (pair >= v.u1 || col >= M) continue;
        const float dg = jb.delta ? jb.delta[pair] : 1.f, du = jb.delta ? jb.delta[F + pair] : 1.f;
        const float gate = bf16_round_f(reduce_at(red, tile, r, col) * dg);
        const float up = bf16_round_f(reduce_at(red, tile, r + 8, col) * du);
        p.act[(size_t)col * F + pair] = __float2bfloat16_rn(gate / (1.0f + expf(-gate)) * up);
      }
      return;
    }
    const int N = jb.N;
    float best = -INFINITY;
    int best_i = 0x7fffffff;
    for (int e = threadIdx.x; e < gt * 16 * 8; e += kThreads) {
      const int r = e & 15, col = (e >> 4) & 7, tile = e >> 7;
      const int n = v.u0 + (tg * GT + tile) * 16 + r;
      if (n >= v.u1 || col >= M) continue;
      const float val = reduce_at(red, tile, r, col) * (jb.delta ? jb.delta[n] : 1.f);
      const size_t idx = (size_t)col * N + n;
      if (jb.kind == kJobQkv) {
        p.qkv[idx] = __float2bfloat16_rn(val);
      } else if (jb.kind == kJobLm) {
        if (p.logits) p.logits[idx] = val;
        // e -> (tile, col, r): a thread sees a single col when kThreads % 128 == 0
        if (val > best || (val == best && n < best_i)) { best = val; best_i = n; }
      } else {  // o / down: residual add into the stream
        const float xv = __bfloat162float(__ldcg(p.x + idx));
        p.x[idx] = __float2bfloat16_rn(bf16_round_f(val) + xv);
      }
    }
    if (jb.kind == kJobLm) {
      // running arg-max of this CTA's vocabulary range: misc[128 + col*2] (value), [.. + 1] (index)
      const int col = (threadIdx.x >> 4) & 7;
      // combine the 16 lanes that share a col (lanes differ in r), then the 4 such groups per col in the CTA
#pragma unroll
      for (int o = 8; o > 0; o >>= 1) {
        const float ob = __shfl_xor_sync(0xffffffffu, best, o);
        const int oi = __shfl_xor_sync(0xffffffffu, best_i, o);
        if (ob > best || (ob == best && oi < best_i)) { best = ob; best_i = oi; }
      }
      float* cand_v = misc + 256;
      int* cand_i = reinterpret_cast<int*>(misc + 256 + 64);
      if ((threadIdx.x & 15) == 0) {
        cand_v[threadIdx.x >> 4] = best;
        cand_i[threadIdx.x >> 4] = best_i;
      }
      __syncthreads();
      if (threadIdx.x < 8) {
        float* run_v = misc + 128;
        int* run_i = reinterpret_cast<int*>(misc + 128 + 8);
        float bv = run_v[threadIdx.x];
        int bi = run_i[threadIdx.x];
        for (int q = 0; q < kThreads / 16; ++q) {
          if (((q & 7) == (int)threadIdx.x)) {
            const float ov = cand_v[q];
            const int oi = cand_i[q];
            if (ov > bv || (ov == bv && oi < bi)) { bv = ov; bi = oi; }
          }
        }
        run_v[threadIdx.x] = bv;
        run_i[threadIdx.x] = bi;
      }
      (void)col;
    }
  }
};

// ---- block bookkeeping + embedding gather (phase 0) -------------------------------------------
__device__ void prep_phase(const MegaParams& p, int cta, int ncta) {
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
  // embedding rows, 16 bytes per thread, spread over the grid
  const int chunks = p.H / 8;
  for (int i = cta * kThreads + threadIdx.x; i < p.M * chunks; i += ncta * kThreads) {
    const int m = i / chunks, c = i % chunks;
    const int tok = p.tokens[m];
    const bool ok = tok >= 0 && tok < p.vocab;
    uint4 v = make_uint4(0, 0, 0, 0);
    if (ok) v = __ldg(reinterpret_cast<const uint4*>(p.embed + (size_t)tok * p.H) + c);
    reinterpret_cast<uint4*>(p.x + (size_t)m * p.H)[c] = v;
  }
}

// ---- attention phase: QK-RMSNorm + RoPE + KV append + split-KV partials -------------------------
template <int D>
__device__ void rope_vec(const __nv_bfloat16* src, const __nv_bfloat16* gain, const float2* rope_row, float eps,
                         __nv_bfloat16* dst, int lane) {
  constexpr int kPairs = D / 64;
  float lo[kPairs], hi[kPairs];
  float ss = 0.f;
#pragma unroll
  for (int q = 0; q < kPairs; ++q) {
    const int d = lane + 32 * q;
    lo[q] = __bfloat162float(__ldcg(src + d));
    hi[q] = __bfloat162float(__ldcg(src + d + D / 2));
    ss += lo[q] * lo[q] + hi[q] * hi[q];
  }
  if (gain != nullptr) {
    ss = warp_sum(ss);
    const float r = 1.0f / sqrtf(ss / (float)D + eps);
#pragma unroll
    for (int q = 0; q < kPairs; ++q) {
      const int d = lane + 32 * q;
      lo[q] = lo[q] * r * __bfloat162float(gain[d]);
      hi[q] = hi[q] * r * __bfloat162float(gain[d + D / 2]);
    }
  }
#pragma unroll
  for (int q = 0; q < kPairs; ++q) {
    const int d = lane + 32 * q;
    const float2 cs = rope_row[d];
    dst[d] = __float2bfloat16_rn(lo[q] * cs.x - hi[q] * cs.y);
    dst[d + D / 2] = __float2bfloat16_rn(hi[q] * cs.x + lo[q] * cs.y);
  }
}

template <int D>
__device__ void attention_phase(const MegaParams& p, int layer, __nv_bfloat16* k_s, __nv_bfloat16* v_s,
                                __nv_bfloat16* q_s, int cta, int ncta) {
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

  for (int item = cta; item < n_items; item += ncta) {
    const int c = item % p.attn_nchunk;
    const int hk = (item / p.attn_nchunk) % p.Hkv;
    const int b = item / (p.attn_nchunk * p.Hkv);
    if (!p.bi.valid[b]) continue;
    const int T = p.block_len[b], P = p.seq_len[b];
    const int Lk = P + T;
    const int key_begin = c * kKeyTile, key_end = min(Lk, key_begin + kKeyTile);
    if (key_begin >= key_end) continue;
    __nv_bfloat16* kbase = kc_l + ((size_t)b * p.Hkv + hk) * (size_t)p.s_max * D;
    __nv_bfloat16* vbase = vc_l + ((size_t)b * p.Hkv + hk) * (size_t)p.s_max * D;
    const int R = G * T;
    __syncthreads();  // shared tiles of the previous item are no longer read

    // (a) rotate this kv head's query rows into shared memory; the item that owns a block row's
    //     cache slot also rotates its K row and stores K and V there
    for (int u = warp; u < R + T; u += NW) {
      if (u < R) {
        const int node = u / G, hq = hk * G + (u % G);
        const int m = b * p.T_max + node;
        rope_vec<D>(p.qkv + (size_t)m * qkv_w + (size_t)hq * D, ly.q_norm,
                    p.rope_table + (size_t)(P + p.bi.depth[m]) * (D / 2), p.rms_eps, q_s + u * kStride, lane);
      } else {
        const int node = u - R;
        const int slot = P + node;
        if (slot >= key_begin && slot < key_end) {
          const int m = b * p.T_max + node;
          rope_vec<D>(p.qkv + (size_t)m * qkv_w + (size_t)(p.Hq + hk) * D, ly.k_norm,
                      p.rope_table + (size_t)(P + p.bi.depth[m]) * (D / 2), p.rms_eps, kbase + (size_t)slot * D, lane);
          const __nv_bfloat16* vsrc = p.qkv + (size_t)m * qkv_w + (size_t)(p.Hq + p.Hkv + hk) * D;
          if (lane < D / 8)
            reinterpret_cast<uint4*>(vbase + (size_t)slot * D)[lane] = __ldcg(reinterpret_cast<const uint4*>(vsrc) + lane);
        }
      }
    }
    __syncthreads();  // block-level visibility of the K/V rows just stored and of q_s

    // (b) stage the K / V tile (zero beyond the end of the sequence)
    for (int i = threadIdx.x; i < kKeyTile * (D / 8); i += kThreads) {
      const int key = i / (D / 8), ch = i % (D / 8);
      uint4 kv4 = make_uint4(0, 0, 0, 0), vv4 = make_uint4(0, 0, 0, 0);
      if (key_begin + key < key_end) {
        kv4 = __ldcg(reinterpret_cast<const uint4*>(kbase + (size_t)(key_begin + key) * D) + ch);
        vv4 = __ldcg(reinterpret_cast<const uint4*>(vbase + (size_t)(key_begin + key) * D) + ch);
      }
      *reinterpret_cast<uint4*>(k_s + key * kStride + ch * 8) = kv4;
      *reinterpret_cast<uint4*>(v_s + key * kStride + ch * 8) = vv4;
    }
    __syncthreads();

    // (c) one warp per 16 query rows
    const int row_tiles = (R + 15) / 16;
    if (warp < row_tiles) {
      uint64_t anc[2];
      uint32_t qf[kDSteps][4];
#pragma unroll
      for (int h = 0; h < 2; ++h) {
        const int r = warp * 16 + g + 8 * h;
        const bool ok = r < R;
        anc[h] = ok ? p.bi.anc[b * p.T_max + r / G] : 0ull;
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
          mma16816(s[j], qf[kd][0], qf[kd][1], qf[kd][2], qf[kd][3], *reinterpret_cast<const uint32_t*>(kr),
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
          if (ok && key >= P) ok = (anc[h] >> (key - P)) & 1ull;
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
      const size_t slot = (((size_t)b * p.Hkv + hk) * p.attn_nchunk + c) * p.attn_rpad;
      // O = P V in two halves of the head dimension (keeps the accumulators within the register budget)
#pragma unroll
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
            mma16816(o[2 * dt], ah[0], ah[1], ah[2], ah[3], b0, b1);
            mma16816(o[2 * dt], al[0], al[1], al[2], al[3], b0, b1);
            mma16816(o[2 * dt + 1], ah[0], ah[1], ah[2], ah[3], b2, b3);
            mma16816(o[2 * dt + 1], al[0], al[1], al[2], al[3], b2, b3);
          }
        }
#pragma unroll
        for (int h = 0; h < 2; ++h) {
          const int r = warp * 16 + g + 8 * h;
          if (r >= p.attn_rpad) continue;
          float* op = p.o_part + (slot + r) * D + half * (D / 2);
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
          p.ml_part[(slot + r) * 2] = row_max[h];
          p.ml_part[(slot + r) * 2 + 1] = row_sum[h];
        }
      }
    }
  }
}

// merge the chunk partials of every (row, query head) in chunk order: one warp per item
template <int D>
__device__ void merge_phase(const MegaParams& p, int cta, int ncta) {
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  constexpr int kPer = D / 32;
  const int G = p.Hq / p.Hkv;
  const int n_items = p.M * p.Hq;
  for (int item = cta * NW + warp; item < n_items; item += ncta * NW) {
    const int hq = item % p.Hq, m = item / p.Hq;
    const int b = m / p.T_max, i = m % p.T_max;
    __nv_bfloat16* dst = p.attn + (size_t)m * p.Hq * D + (size_t)hq * D;
    if (!p.bi.valid[b] || i >= p.block_len[b]) {
#pragma unroll
      for (int e = 0; e < kPer; ++e) dst[lane * kPer + e] = __float2bfloat16_rn(0.f);
      continue;
    }
    const int hk = hq / G, r = i * G + (hq % G);
    const int Lk = p.seq_len[b] + p.block_len[b];
    const int nch = (Lk + kKeyTile - 1) / kKeyTile;
    const size_t slot0 = ((size_t)b * p.Hkv + hk) * p.attn_nchunk * p.attn_rpad;
    float mx = -INFINITY;
    for (int c = lane; c < nch; c += 32) mx = fmaxf(mx, __ldcg(p.ml_part + (slot0 + (size_t)c * p.attn_rpad + r) * 2));
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) mx = fmaxf(mx, __shfl_xor_sync(0xffffffffu, mx, o));
    float acc[kPer];
#pragma unroll
    for (int e = 0; e < kPer; ++e) acc[e] = 0.f;
    float den = 0.f;
    for (int c = 0; c < nch; ++c) {
      const size_t s = slot0 + (size_t)c * p.attn_rpad + r;
      const float2 ml = __ldcg(reinterpret_cast<const float2*>(p.ml_part + s * 2));
      if (ml.x == -INFINITY) continue;
      const float w = exp2f(ml.x - mx);
      den += w * ml.y;
      if constexpr (kPer == 4) {
        const float4 ov = __ldcg(reinterpret_cast<const float4*>(p.o_part + s * D) + lane);
        acc[0] += w * ov.x; acc[1] += w * ov.y; acc[2] += w * ov.z; acc[kPer - 1] += w * ov.w;
      } else {
        const float2 ov = __ldcg(reinterpret_cast<const float2*>(p.o_part + s * D) + lane);
        acc[0] += w * ov.x; acc[kPer - 1] += w * ov.y;
      }
    }
    const float inv = 1.0f / den;
#pragma unroll
    for (int e = 0; e < kPer; ++e) dst[lane * kPer + e] = __float2bfloat16_rn(acc[e] * inv);
  }
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
  __syncthreads();
  if ((int)threadIdx.x < p.B) {
    const int b = threadIdx.x, base = b * p.T_max;
    if (!p.bi.valid[b]) {
      p.accept_len[b] = 0;
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
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  unsigned char* ring = smem + (size_t)warp * kStages * kStageBytes;
  unsigned char* uni = smem + kRingBytes;
  float* red = reinterpret_cast<float*>(uni);
  __nv_bfloat16* k_s = reinterpret_cast<__nv_bfloat16*>(uni);
  __nv_bfloat16* v_s = reinterpret_cast<__nv_bfloat16*>(uni + kKvTileBytes);
  __nv_bfloat16* q_s = reinterpret_cast<__nv_bfloat16*>(uni + kUnionBytes);
  float* misc = reinterpret_cast<float*>(uni + kUnionBytes + kQTileBytes);
  int* abort_flag = reinterpret_cast<int*>(misc + 200);

  if (threadIdx.x == 0) *abort_flag = 0;
  if (threadIdx.x < 8) {  // running arg-max of this CTA
    misc[128 + threadIdx.x] = -INFINITY;
    reinterpret_cast<int*>(misc + 128 + 8)[threadIdx.x] = 0x7fffffff;
  }
  __syncthreads();

  // start the weight stream: the first kStages-1 stages of this warp's schedule
  Producer<W_INT8> prod;
  prod.init(p.jobs, p.n_jobs, cta, ncta, warp, lane);
  unsigned cstage = 0;
#pragma unroll 1
  for (int s = 0; s < kStages - 1; ++s) prod.fetch(ring + s * kStageBytes);

  GridSync gs{p.barrier, p.status, (unsigned)ncta, 0u, abort_flag};
  bool ok = true;

  prep_phase(p, cta, ncta);
  ok = gs.sync();
  for (int l = 0; l < p.L && ok; ++l) {
    GemmPhase<W_INT8>::run(p, 4 * l + 0, prod, ring, cstage, red, misc, cta, ncta);
    if (!(ok = gs.sync())) break;
    attention_phase<D>(p, l, k_s, v_s, q_s, cta, ncta);
    if (!(ok = gs.sync())) break;
    merge_phase<D>(p, cta, ncta);
    if (!(ok = gs.sync())) break;
    GemmPhase<W_INT8>::run(p, 4 * l + 1, prod, ring, cstage, red, misc, cta, ncta);
    if (!(ok = gs.sync())) break;
    GemmPhase<W_INT8>::run(p, 4 * l + 2, prod, ring, cstage, red, misc, cta, ncta);
    if (!(ok = gs.sync())) break;
    GemmPhase<W_INT8>::run(p, 4 * l + 3, prod, ring, cstage, red, misc, cta, ncta);
    if (!(ok = gs.sync())) break;
  }
  if (ok) {
    GemmPhase<W_INT8>::run(p, 4 * p.L, prod, ring, cstage, red, misc, cta, ncta);
    __syncthreads();
    if (threadIdx.x < 8) {
      p.cand_val[(size_t)cta * 8 + threadIdx.x] = misc[128 + threadIdx.x];
      p.cand_idx[(size_t)cta * 8 + threadIdx.x] = reinterpret_cast<int*>(misc + 128 + 8)[threadIdx.x];
    }
    ok = gs.sync();
    if (ok && cta == 0) accept_phase(p, ncta);
  }
  cp_async_wait<0>();  // nothing of ours is in flight when the CTA leaves
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
