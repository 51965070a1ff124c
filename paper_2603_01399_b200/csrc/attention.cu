// Grouped-query verify-attention (the attention of the verification pass, Section 3.1:
// every block row attends to the cached context x_<t plus the block rows its mask allows —
// earlier rows for a chain, ancestors for a tree).
//
// The second HBM stream of the pass: K and V of the prefix are read once per layer
// (2 * 2 B * D per cached position per kv head).  One kv head serves R = G * T query rows
// (G = Hq / Hkv query heads x T block rows; 24..85 here), i.e. 2R flop per K/V byte, which
// is far above what FMA pipes sustain at HBM speed, so QK^T and PV run on the tensor
// cores (mma.m16n8k16, bf16 in, fp32 accumulate) with the softmax in registers and
// warp-shuffle row reductions.
//
// Parallelism: the key range of a sequence is cut into chunks of `chunk` positions; a CTA
// handles one (sequence, kv head, chunk) with one warp per 16 query rows, all warps
// sharing the K/V tiles staged in shared memory.  Each CTA leaves an un-normalised partial
// (row max, row sum, O) and a second kernel merges the partials of a row in chunk order.
// P is fed to the PV product as a bf16 high part plus a bf16 low part (two MMAs), which
// keeps ~16 bits of the probabilities.
#include <math.h>

#include "common.cuh"

namespace quasar {

namespace {

constexpr int kKeyTile = 32;   // keys staged in shared memory at a time
constexpr int kMaxWarps = 3;   // per CTA; four CTAs share an SM (168 registers per thread, 35 KB of tiles)
constexpr float kLog2e = 1.4426950408889634f;

struct AttnArgs {
  const __nv_bfloat16* qkv;  // [B*T_max][(Hq+2Hkv)*D], q part already normalised + rotated
  const __nv_bfloat16* kc;   // [B][Hkv][s_max][D]
  const __nv_bfloat16* vc;
  const int32_t* seq_len;
  const int32_t* block_len;
  BlockInfo bi;
  float* o_part;             // [B][Hkv][nchunk][Rpad][D]
  float* ml_part;            // [B][Hkv][nchunk][Rpad][2]
  __nv_bfloat16* out;        // [B*T_max][Hq*D]
  int B, T_max, Hq, Hkv, s_max, chunk, nchunk, Rpad, ngroups;
};

__device__ __forceinline__ void mma16816(float (&c)[4], uint32_t a0, uint32_t a1, uint32_t a2, uint32_t a3,
                                         uint32_t b0, uint32_t b1) {
  asm("mma.sync.aligned.m16n8k16.row.col.f32.bf16.bf16.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%0,%1,%2,%3};\n"
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

__device__ __forceinline__ void ldmatrix_x4(uint32_t& r0, uint32_t& r1, uint32_t& r2, uint32_t& r3, const void* smem_ptr) {
  const uint32_t addr = (uint32_t)__cvta_generic_to_shared(smem_ptr);
  asm volatile("ldmatrix.sync.aligned.m8n8.x4.shared.b16 {%0,%1,%2,%3}, [%4];\n"
               : "=r"(r0), "=r"(r1), "=r"(r2), "=r"(r3)
               : "r"(addr));
}

__device__ __forceinline__ uint32_t pack_bf16(float lo, float hi) {
  __nv_bfloat162 p = __floats2bfloat162_rn(lo, hi);
  return *reinterpret_cast<uint32_t*>(&p);
}

// high and low bf16 parts of a pair of probabilities
__device__ __forceinline__ void split_bf16(float a, float b, uint32_t& hi, uint32_t& lo) {
  const __nv_bfloat16 ah = __float2bfloat16_rn(a), bh = __float2bfloat16_rn(b);
  const float ar = a - __bfloat162float(ah), br = b - __bfloat162float(bh);
  __nv_bfloat162 h;
  h.x = ah;
  h.y = bh;
  hi = *reinterpret_cast<uint32_t*>(&h);
  lo = pack_bf16(ar, br);
}

template <int D>
__global__ void __launch_bounds__(kMaxWarps * 32, 4) verify_attention_kernel(AttnArgs a) {
  constexpr int kStride = D + 8;  // padded row of the staged K / V tiles (bf16 elements)
  constexpr int kDSteps = D / 16;
  // two K tiles and two V tiles: the next tile of the chunk lands (cp.async) while the current one is multiplied
  extern __shared__ __align__(16) unsigned char attn_smem[];
  __nv_bfloat16* const tiles = reinterpret_cast<__nv_bfloat16*>(attn_smem);
  constexpr int kTileElems = kKeyTile * kStride;

  const int c = blockIdx.x / a.ngroups, group = blockIdx.x % a.ngroups;
  const int hk = blockIdx.y, b = blockIdx.z;
  if (!a.bi.valid[b]) return;
  const int T = a.block_len[b];
  const int P = a.seq_len[b];
  const int Lk = P + T;
  const int key_begin = c * a.chunk;
  const int key_end = min(Lk, key_begin + a.chunk);
  if (key_begin >= key_end) return;

  const int G = a.Hq / a.Hkv;
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int nwarps = blockDim.x >> 5;
  const int g = lane >> 2, t = lane & 3;
  const int row_tile = group * nwarps + warp;
  const int qkv_w = (a.Hq + 2 * a.Hkv) * D;

  // the two query rows of this thread: r = node * G + head-in-group
  int node[2];
  uint64_t anc[2];
  uint32_t qf[kDSteps][4];
#pragma unroll
  for (int h = 0; h < 2; ++h) {
    const int r = row_tile * 16 + g + 8 * h;
    node[h] = r / G;
    const bool ok = node[h] < T;
    anc[h] = ok ? a.bi.anc[b * a.T_max + node[h]] : 0ull;
    const __nv_bfloat16* qrow =
        a.qkv + (size_t)(b * a.T_max + (ok ? node[h] : 0)) * qkv_w + (size_t)(hk * G + (r % G)) * D;
#pragma unroll
    for (int kd = 0; kd < kDSteps; ++kd) {
      qf[kd][h] = ok ? *reinterpret_cast<const uint32_t*>(qrow + kd * 16 + 2 * t) : 0u;
      qf[kd][h + 2] = ok ? *reinterpret_cast<const uint32_t*>(qrow + kd * 16 + 8 + 2 * t) : 0u;
    }
  }

  float o[D / 8][4];
#pragma unroll
  for (int i = 0; i < D / 8; ++i) o[i][0] = o[i][1] = o[i][2] = o[i][3] = 0.f;
  float row_max[2] = {-INFINITY, -INFINITY};
  float row_sum[2] = {0.f, 0.f};
  const float scale_log2 = kLog2e / sqrtf((float)D);

  const __nv_bfloat16* kbase = a.kc + ((size_t)b * a.Hkv + hk) * (size_t)a.s_max * D;
  const __nv_bfloat16* vbase = a.vc + ((size_t)b * a.Hkv + hk) * (size_t)a.s_max * D;

  // the cached K / V rows are read once per pass: evict-first in L2
  uint64_t kv_policy;
  asm volatile("createpolicy.fractional.L2::evict_first.b64 %0, 1.0;\n" : "=l"(kv_policy));
  auto stage_tile = [&](int buf, int k0) {
    __nv_bfloat16* kd = tiles + buf * 2 * kTileElems;
    __nv_bfloat16* vd = kd + kTileElems;
    for (int i = threadIdx.x; i < kKeyTile * (D / 8); i += blockDim.x) {
      const int key = i / (D / 8), ch = i % (D / 8);
      if (k0 + key < key_end) {
        const uint32_t ks = (uint32_t)__cvta_generic_to_shared(kd + key * kStride + ch * 8);
        const uint32_t vs = (uint32_t)__cvta_generic_to_shared(vd + key * kStride + ch * 8);
        asm volatile("cp.async.cg.shared.global.L2::cache_hint [%0], [%1], 16, %2;\n" ::"r"(ks), "l"(kbase + (size_t)(k0 + key) * D + ch * 8), "l"(kv_policy) : "memory");
        asm volatile("cp.async.cg.shared.global.L2::cache_hint [%0], [%1], 16, %2;\n" ::"r"(vs), "l"(vbase + (size_t)(k0 + key) * D + ch * 8), "l"(kv_policy) : "memory");
      } else {
        *reinterpret_cast<uint4*>(kd + key * kStride + ch * 8) = make_uint4(0, 0, 0, 0);
        *reinterpret_cast<uint4*>(vd + key * kStride + ch * 8) = make_uint4(0, 0, 0, 0);
      }
    }
    asm volatile("cp.async.commit_group;\n" ::: "memory");
  };
  stage_tile(0, key_begin);
  int buf = 0;
  for (int k0 = key_begin; k0 < key_end; k0 += kKeyTile, buf ^= 1) {
    if (k0 + kKeyTile < key_end) {
      stage_tile(buf ^ 1, k0 + kKeyTile);           // (its last readers passed the barrier that ended the tile before)
      asm volatile("cp.async.wait_group 1;\n" ::: "memory");
    } else {
      asm volatile("cp.async.wait_group 0;\n" ::: "memory");
    }
    __syncthreads();
    const __nv_bfloat16* k_s = tiles + buf * 2 * kTileElems;
    const __nv_bfloat16* v_s = k_s + kTileElems;

    // S = Q K^T for 16 rows x 64 keys.  One ldmatrix brings the K fragments of 8 keys x 32 head dimensions;
    // MMAs on the same accumulator are kept apart (a dependent MMA waits ~20 cycles).
    float s[kKeyTile / 8][4];
#pragma unroll
    for (int j = 0; j < kKeyTile / 8; ++j) s[j][0] = s[j][1] = s[j][2] = s[j][3] = 0.f;
    {
      const __nv_bfloat16* k_lane = k_s + (lane & 7) * kStride + (lane >> 3) * 8;
#pragma unroll
      for (int kd2 = 0; kd2 < kDSteps / 2; ++kd2) {
#pragma unroll
        for (int jp = 0; jp < kKeyTile / 16; ++jp) {
          uint32_t ka[4], kb[4];
          ldmatrix_x4(ka[0], ka[1], ka[2], ka[3], k_lane + (16 * jp) * kStride + kd2 * 32);
          ldmatrix_x4(kb[0], kb[1], kb[2], kb[3], k_lane + (16 * jp + 8) * kStride + kd2 * 32);
          mma16816(s[2 * jp], qf[2 * kd2][0], qf[2 * kd2][1], qf[2 * kd2][2], qf[2 * kd2][3], ka[0], ka[1]);
          mma16816(s[2 * jp + 1], qf[2 * kd2][0], qf[2 * kd2][1], qf[2 * kd2][2], qf[2 * kd2][3], kb[0], kb[1]);
          mma16816(s[2 * jp], qf[2 * kd2 + 1][0], qf[2 * kd2 + 1][1], qf[2 * kd2 + 1][2], qf[2 * kd2 + 1][3], ka[2], ka[3]);
          mma16816(s[2 * jp + 1], qf[2 * kd2 + 1][0], qf[2 * kd2 + 1][1], qf[2 * kd2 + 1][2], qf[2 * kd2 + 1][3], kb[2], kb[3]);
        }
      }
    }

    // mask, running max
    float tile_max[2] = {-INFINITY, -INFINITY};
#pragma unroll
    for (int j = 0; j < kKeyTile / 8; ++j) {
#pragma unroll
      for (int e = 0; e < 4; ++e) {
        const int h = e >> 1;
        const int key = k0 + 8 * j + 2 * t + (e & 1);
        bool ok = key < key_end;
        if (ok && key >= P) ok = (anc[h] >> (key - P)) & 1ull;
        const float v = ok ? s[j][e] * scale_log2 : -INFINITY;
        s[j][e] = v;
        tile_max[h] = fmaxf(tile_max[h], v);
      }
    }
    float alpha[2], m_use[2];
#pragma unroll
    for (int h = 0; h < 2; ++h) {
      tile_max[h] = fmaxf(tile_max[h], __shfl_xor_sync(0xffffffffu, tile_max[h], 1));
      tile_max[h] = fmaxf(tile_max[h], __shfl_xor_sync(0xffffffffu, tile_max[h], 2));
      const float m_new = fmaxf(row_max[h], tile_max[h]);
      m_use[h] = (m_new == -INFINITY) ? 0.f : m_new;
      alpha[h] = exp2f(row_max[h] - m_use[h]);  // 0 when nothing has been seen yet
      row_max[h] = m_new;
      row_sum[h] *= alpha[h];
    }
#pragma unroll
    for (int i = 0; i < D / 8; ++i) {
      o[i][0] *= alpha[0];
      o[i][1] *= alpha[0];
      o[i][2] *= alpha[1];
      o[i][3] *= alpha[1];
    }
#pragma unroll
    for (int j = 0; j < kKeyTile / 8; ++j) {
#pragma unroll
      for (int e = 0; e < 4; ++e) {
        const float p = exp2f(s[j][e] - m_use[e >> 1]);
        s[j][e] = p;
        row_sum[e >> 1] += p;
      }
    }

    // O += P V, 16 keys per step
#pragma unroll
    for (int kk = 0; kk < kKeyTile / 16; ++kk) {
      uint32_t ah[4], al[4];
      split_bf16(s[2 * kk][0], s[2 * kk][1], ah[0], al[0]);
      split_bf16(s[2 * kk][2], s[2 * kk][3], ah[1], al[1]);
      split_bf16(s[2 * kk + 1][0], s[2 * kk + 1][1], ah[2], al[2]);
      split_bf16(s[2 * kk + 1][2], s[2 * kk + 1][3], ah[3], al[3]);
#pragma unroll
      for (int dt = 0; dt < D / 16; dt += 2) {
        uint32_t b[2][4];
        const int mat = lane >> 3, r = lane & 7;
        const __nv_bfloat16* v_lane = v_s + (kk * 16 + (mat & 1) * 8 + r) * kStride + (mat >> 1) * 8;
        ldmatrix_x4_trans(b[0][0], b[0][1], b[0][2], b[0][3], v_lane + dt * 16);
        ldmatrix_x4_trans(b[1][0], b[1][1], b[1][2], b[1][3], v_lane + dt * 16 + 16);
        mma16816(o[2 * dt], ah[0], ah[1], ah[2], ah[3], b[0][0], b[0][1]);
        mma16816(o[2 * dt + 1], ah[0], ah[1], ah[2], ah[3], b[0][2], b[0][3]);
        mma16816(o[2 * dt + 2], ah[0], ah[1], ah[2], ah[3], b[1][0], b[1][1]);
        mma16816(o[2 * dt + 3], ah[0], ah[1], ah[2], ah[3], b[1][2], b[1][3]);
        mma16816(o[2 * dt], al[0], al[1], al[2], al[3], b[0][0], b[0][1]);
        mma16816(o[2 * dt + 1], al[0], al[1], al[2], al[3], b[0][2], b[0][3]);
        mma16816(o[2 * dt + 2], al[0], al[1], al[2], al[3], b[1][0], b[1][1]);
        mma16816(o[2 * dt + 3], al[0], al[1], al[2], al[3], b[1][2], b[1][3]);
      }
    }
    __syncthreads();   // every warp is done with this tile before the copy of the tile after next overwrites it
  }

  // ---- partial results ----------------------------------------------------------------------
#pragma unroll
  for (int h = 0; h < 2; ++h) {
    row_sum[h] += __shfl_xor_sync(0xffffffffu, row_sum[h], 1);
    row_sum[h] += __shfl_xor_sync(0xffffffffu, row_sum[h], 2);
  }
  const size_t slot = (((size_t)b * a.Hkv + hk) * a.nchunk + c) * a.Rpad;
#pragma unroll
  for (int h = 0; h < 2; ++h) {
    const int r = row_tile * 16 + g + 8 * h;
    if (r >= a.Rpad) continue;
    float* op = a.o_part + (slot + r) * D;
#pragma unroll
    for (int i = 0; i < D / 8; ++i) {
      *reinterpret_cast<float2*>(op + 8 * i + 2 * t) = make_float2(o[i][2 * h], o[i][2 * h + 1]);
    }
    if (t == 0) {
      a.ml_part[(slot + r) * 2] = row_max[h];
      a.ml_part[(slot + r) * 2 + 1] = row_sum[h];
    }
  }
}

// One warp per (sequence, block row, query head): merge the chunk partials in chunk order.
template <int D>
__global__ void __launch_bounds__(128) attention_merge_kernel(AttnArgs a) {
  const int item = blockIdx.x * 4 + (threadIdx.x >> 5);
  const int lane = threadIdx.x & 31;
  if (item >= a.B * a.T_max * a.Hq) return;
  const int hq = item % a.Hq;
  const int m = item / a.Hq;
  const int b = m / a.T_max, i = m % a.T_max;
  __nv_bfloat16* dst = a.out + (size_t)m * a.Hq * D + (size_t)hq * D;
  constexpr int kPer = D / 32;
  if (!a.bi.valid[b] || i >= a.block_len[b]) {
#pragma unroll
    for (int e = 0; e < kPer; ++e) dst[lane * kPer + e] = __float2bfloat16_rn(0.f);
    return;
  }
  const int G = a.Hq / a.Hkv;
  const int hk = hq / G;
  const int r = i * G + (hq % G);
  const int Lk = a.seq_len[b] + a.block_len[b];
  const int nch = (Lk + a.chunk - 1) / a.chunk;
  const size_t slot0 = ((size_t)b * a.Hkv + hk) * a.nchunk * a.Rpad;
  // the row's maximum over the chunks: the lanes take the chunks in turn
  float mx = -INFINITY;
  for (int c = lane; c < nch; c += 32) mx = fmaxf(mx, a.ml_part[(slot0 + (size_t)c * a.Rpad + r) * 2]);
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) mx = fmaxf(mx, __shfl_xor_sync(0xffffffffu, mx, o));
  float acc[kPer];
#pragma unroll
  for (int e = 0; e < kPer; ++e) acc[e] = 0.f;
  float den = 0.f;
  // chunks are added in chunk order, eight at a time so that their loads are in flight together
  for (int c0 = 0; c0 < nch; c0 += 8) {
    float2 ml[8];
    float ov[8][kPer];
#pragma unroll
    for (int j = 0; j < 8; ++j) {
      const bool in = c0 + j < nch;
      const size_t s = slot0 + (size_t)(in ? c0 + j : c0) * a.Rpad + r;
      ml[j] = in ? *reinterpret_cast<const float2*>(a.ml_part + s * 2) : make_float2(-INFINITY, 0.f);
      if constexpr (kPer == 4) {
        const float4 v = *reinterpret_cast<const float4*>(a.o_part + s * D + lane * kPer);
        ov[j][0] = v.x; ov[j][1] = v.y; ov[j][2] = v.z; ov[j][3] = v.w;
      } else {
        const float2 v = *reinterpret_cast<const float2*>(a.o_part + s * D + lane * kPer);
        ov[j][0] = v.x; ov[j][1] = v.y;
      }
    }
#pragma unroll
    for (int j = 0; j < 8; ++j) {
      if (ml[j].x == -INFINITY) continue;
      const float w = exp2f(ml[j].x - mx);
      den += w * ml[j].y;
#pragma unroll
      for (int e = 0; e < kPer; ++e) acc[e] += w * ov[j][e];
    }
  }
  const float inv = 1.0f / den;
#pragma unroll
  for (int e = 0; e < kPer; ++e) dst[lane * kPer + e] = __float2bfloat16_rn(acc[e] * inv);
}

struct AttnPlan {
  int chunk, nchunk, Rpad, ngroups, warps;
};

AttnPlan plan_attention(int B, int T_max, int Hq, int Hkv, int s_max) {
  AttnPlan p;
  const int units = B * Hkv;
  int per_unit = (2 * 148 + units - 1) / units;
  if (per_unit < 1) per_unit = 1;
  int chunk = (s_max + per_unit - 1) / per_unit;
  chunk = (chunk + kKeyTile - 1) / kKeyTile * kKeyTile;
  if (chunk < kKeyTile) chunk = kKeyTile;
  if (chunk > 256) chunk = 256;
  p.chunk = chunk;
  p.nchunk = (s_max + chunk - 1) / chunk;
  const int R = (Hq / Hkv) * T_max;
  const int tiles = (R + 15) / 16;
  p.ngroups = (tiles + kMaxWarps - 1) / kMaxWarps;
  p.warps = (tiles + p.ngroups - 1) / p.ngroups;
  p.Rpad = p.ngroups * p.warps * 16;
  return p;
}

}  // namespace

size_t attention_workspace_bytes(int B, int T_max, int Hq, int Hkv, int D, int s_max) {
  const AttnPlan p = plan_attention(B, T_max, Hq, Hkv, s_max);
  const size_t rows = (size_t)B * Hkv * p.nchunk * p.Rpad;
  return rows * D * sizeof(float) + rows * 2 * sizeof(float);
}

int launch_attention(const __nv_bfloat16* qkv, const __nv_bfloat16* k_cache_layer, const __nv_bfloat16* v_cache_layer,
                     const int32_t* seq_len, const int32_t* block_len, BlockInfo bi, int B, int T_max, int Hq, int Hkv,
                     int D, int s_max, __nv_bfloat16* out, void* workspace, size_t workspace_bytes,
                     cudaStream_t stream) {
  const AttnPlan p = plan_attention(B, T_max, Hq, Hkv, s_max);
  if (workspace_bytes < attention_workspace_bytes(B, T_max, Hq, Hkv, D, s_max)) {
    set_error("attention: workspace too small");
    return QUASAR_ERR_CAPACITY;
  }
  AttnArgs a;
  a.qkv = qkv; a.kc = k_cache_layer; a.vc = v_cache_layer; a.seq_len = seq_len; a.block_len = block_len; a.bi = bi;
  const size_t rows = (size_t)B * Hkv * p.nchunk * p.Rpad;
  a.o_part = reinterpret_cast<float*>(workspace);
  a.ml_part = a.o_part + rows * D;
  a.out = out;
  a.B = B; a.T_max = T_max; a.Hq = Hq; a.Hkv = Hkv; a.s_max = s_max;
  a.chunk = p.chunk; a.nchunk = p.nchunk; a.Rpad = p.Rpad; a.ngroups = p.ngroups;
  dim3 grid(p.nchunk * p.ngroups, Hkv, B);
  const int items = B * T_max * Hq;
  if (D == 128) {
    constexpr size_t smem128 = 4u * kKeyTile * (128 + 8) * sizeof(__nv_bfloat16);
    static bool configured128 = false;
    if (!configured128) {
      QUASAR_CUDA_CHECK(cudaFuncSetAttribute(verify_attention_kernel<128>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem128));
      QUASAR_CUDA_CHECK(cudaFuncSetAttribute(verify_attention_kernel<128>, cudaFuncAttributePreferredSharedMemoryCarveout, 100));
      configured128 = true;
    }
    verify_attention_kernel<128><<<grid, p.warps * 32, smem128, stream>>>(a);
    QUASAR_LAUNCH_CHECK();
    attention_merge_kernel<128><<<(items + 3) / 4, 128, 0, stream>>>(a);
    QUASAR_LAUNCH_CHECK();
  } else if (D == 64) {
    constexpr size_t smem64 = 4u * kKeyTile * (64 + 8) * sizeof(__nv_bfloat16);
    verify_attention_kernel<64><<<grid, p.warps * 32, smem64, stream>>>(a);
    QUASAR_LAUNCH_CHECK();
    attention_merge_kernel<64><<<(items + 3) / 4, 128, 0, stream>>>(a);
    QUASAR_LAUNCH_CHECK();
  } else {
    set_error("head_dim %d not supported (64 or 128)", D);
    return QUASAR_ERR_SHAPE;
  }
  return QUASAR_OK;
}

}  // namespace quasar
