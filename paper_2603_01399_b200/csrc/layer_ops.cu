// The small steps around the GEMMs of the verification pass (Section 3.3: the "non-linear
// layers" that stay in high precision): block bookkeeping, embedding gather, RMSNorm,
// QK-RMSNorm + RoPE + KV append, SwiGLU, arg-max, greedy acceptance (Section 3.1 Eq. 2 at
// temperature 0) and the cache commit.  All are HBM/L2-bound on a few KB..MB; fp32 math,
// bf16 storage.
#include <math.h>

#include <cuda_fp16.h>

#include "common.cuh"

namespace quasar {

namespace {

__device__ __forceinline__ float warp_sum(float v) {
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
  return v;
}

// ---- block bookkeeping -------------------------------------------------------------------
// One thread per sequence: checks tokens / parents / capacity, derives ancestor bit masks and depths.
__global__ void block_prep_kernel(const int32_t* __restrict__ tokens, const int32_t* __restrict__ parents,
                                  const int32_t* __restrict__ block_len, const int32_t* __restrict__ seq_len, int B,
                                  int T_max, int s_max, int vocab, BlockInfo bi, int32_t* status) {
  const int b = blockIdx.x * blockDim.x + threadIdx.x;
  if (b >= B) return;
  const int T = block_len[b];
  const int P = seq_len[b];
  int err = 0;
  if (T < 1 || T > T_max || P < 0) err = QUASAR_ERR_INVALID_ARG;
  else if (P + T > s_max) err = QUASAR_ERR_CAPACITY;
  if (!err) {
    for (int i = 0; i < T; ++i) {
      const int tok = tokens[b * T_max + i];
      if (tok < 0 || tok >= vocab) err = QUASAR_ERR_TOKEN;
      int p = (parents == nullptr) ? i - 1 : parents[b * T_max + i];
      if ((i == 0 && p != -1) || (i > 0 && (p < 0 || p >= i))) err = QUASAR_ERR_TREE;
      if (err) break;
      uint64_t m = 1ull << i;
      int d = 0;
      if (i > 0) {
        m |= bi.anc[b * T_max + p];
        d = bi.depth[b * T_max + p] + 1;
      }
      bi.anc[b * T_max + i] = m;
      bi.depth[b * T_max + i] = d;
    }
  }
  for (int i = (err ? 0 : T); i < T_max; ++i) {
    bi.anc[b * T_max + i] = 0;
    bi.depth[b * T_max + i] = 0;
  }
  bi.valid[b] = err ? 0 : 1;
  if (err && status) atomicMin(status, err);
}

// ---- embedding gather ----------------------------------------------------------------------
__global__ void embed_kernel(const int32_t* __restrict__ tokens, const __nv_bfloat16* __restrict__ embed, int H,
                             int vocab, __nv_bfloat16* __restrict__ x) {
  const int m = blockIdx.x;
  int tok = tokens[m];
  const bool ok = tok >= 0 && tok < vocab;
  const uint4* src = reinterpret_cast<const uint4*>(embed + (size_t)(ok ? tok : 0) * H);
  uint4* dst = reinterpret_cast<uint4*>(x + (size_t)m * H);
  for (int i = threadIdx.x; i < H / 8; i += blockDim.x) dst[i] = ok ? __ldg(src + i) : make_uint4(0, 0, 0, 0);
}

// ---- RMSNorm: y = x * rsqrt(mean(x^2) + eps) * g ------------------------------------------
__global__ void __launch_bounds__(256)
rmsnorm_kernel(const __nv_bfloat16* __restrict__ x, const __nv_bfloat16* __restrict__ g, int H, float eps,
               __nv_bfloat16* __restrict__ y) {
  const int m = blockIdx.x;
  const __nv_bfloat162* xr = reinterpret_cast<const __nv_bfloat162*>(x + (size_t)m * H);
  const __nv_bfloat162* gr = reinterpret_cast<const __nv_bfloat162*>(g);
  __nv_bfloat162* yr = reinterpret_cast<__nv_bfloat162*>(y + (size_t)m * H);
  float ss = 0.f;
  for (int i = threadIdx.x; i < H / 2; i += blockDim.x) {
    const float2 f = __bfloat1622float2(xr[i]);
    ss += f.x * f.x + f.y * f.y;
  }
  ss = warp_sum(ss);
  __shared__ float s_part[8];
  if ((threadIdx.x & 31) == 0) s_part[threadIdx.x >> 5] = ss;
  __syncthreads();
  float tot = 0.f;
#pragma unroll
  for (int i = 0; i < 8; ++i) tot += s_part[i];
  const float r = 1.0f / sqrtf(tot / (float)H + eps);
  for (int i = threadIdx.x; i < H / 2; i += blockDim.x) {
    const float2 f = __bfloat1622float2(xr[i]);
    const float2 gg = __bfloat1622float2(gr[i]);
    yr[i] = __floats2bfloat162_rn(f.x * r * gg.x, f.y * r * gg.y);
  }
}

// One thread block per activation row would leave half the SMs idle and every thread with a long chain of
// dependent round trips to L2, so these row kernels run 1024 threads per row.
constexpr int kRowThreads = 1024;

// block-wide maximum of non-negative values
__device__ __forceinline__ float block_max_rows(float v, float* s_buf) {
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) v = fmaxf(v, __shfl_xor_sync(0xffffffffu, v, o));
  __syncthreads();
  if ((threadIdx.x & 31) == 0) s_buf[threadIdx.x >> 5] = v;
  __syncthreads();
  float r = s_buf[0];
#pragma unroll
  for (int i = 1; i < kRowThreads / 32; ++i) r = fmaxf(r, s_buf[i]);
  return r;
}

// A row stays in registers between its passes: thread t holds the pairs t, t + 1024, ... (at most kNormPairs of them,
// i.e. rows of up to 8192 elements; the launcher refuses longer ones).
constexpr int kNormPairs = 4;

template <bool REDUCE>
__global__ void __launch_bounds__(kRowThreads)
rmsnorm_f16_kernel(const float* __restrict__ partial, int nsplit, int mpad, const float* __restrict__ dx,
                   const float* __restrict__ dw, __nv_bfloat16* __restrict__ x, const __nv_bfloat16* __restrict__ g, int H,
                   float eps, __nv_bfloat16* __restrict__ y, __half* __restrict__ y16, float* __restrict__ inv) {
  const int m = blockIdx.x;
  __nv_bfloat162* xr = reinterpret_cast<__nv_bfloat162*>(x + (size_t)m * H);
  const __nv_bfloat162* gr = reinterpret_cast<const __nv_bfloat162*>(g);
  __nv_bfloat162* yr = reinterpret_cast<__nv_bfloat162*>(y + (size_t)m * H);
  __half2* hr = reinterpret_cast<__half2*>(y16 + (size_t)m * H);
  __shared__ float s_part[kRowThreads / 32];
  const int np = H / 2;
  float2 xv[kNormPairs], gv[kNormPairs];
  float ss = 0.f;
#pragma unroll
  for (int j = 0; j < kNormPairs; ++j) {
    const int i = threadIdx.x + j * kRowThreads;
    xv[j] = make_float2(0.f, 0.f);
    gv[j] = make_float2(0.f, 0.f);
    if (i < np) {
      gv[j] = __bfloat1622float2(gr[i]);
      if (REDUCE) {
        const float dxm = dx[m];
        const size_t split_stride = (size_t)mpad * H;
        const float* p0 = partial + (size_t)m * H;
        float2 acc = make_float2(0.f, 0.f);
        for (int sp = 0; sp < nsplit; ++sp) {   // k-ranges in ascending order
          const float2 v = __ldcg(reinterpret_cast<const float2*>(p0 + (size_t)sp * split_stride) + i);
          acc.x += v.x;
          acc.y += v.y;
        }
        const float2 d = *reinterpret_cast<const float2*>(dw + 2 * i);
        const float2 r = __bfloat1622float2(xr[i]);
        const float v0 = __bfloat162float(__float2bfloat16_rn((acc.x * dxm) * d.x)) + r.x;
        const float v1 = __bfloat162float(__float2bfloat16_rn((acc.y * dxm) * d.y)) + r.y;
        const __nv_bfloat162 o = __floats2bfloat162_rn(v0, v1);
        xr[i] = o;
        xv[j] = __bfloat1622float2(o);
      } else {
        xv[j] = __bfloat1622float2(xr[i]);
      }
      ss += xv[j].x * xv[j].x + xv[j].y * xv[j].y;
    }
  }
  ss = warp_sum(ss);
  if ((threadIdx.x & 31) == 0) s_part[threadIdx.x >> 5] = ss;
  __syncthreads();
  float tot = 0.f;
#pragma unroll
  for (int i = 0; i < kRowThreads / 32; ++i) tot += s_part[i];
  const float r = 1.0f / sqrtf(tot / (float)H + eps);
  float amax = 0.f;
#pragma unroll
  for (int j = 0; j < kNormPairs; ++j) {
    const int i = threadIdx.x + j * kRowThreads;
    if (i < np) {
      const __nv_bfloat162 o = __floats2bfloat162_rn(xv[j].x * r * gv[j].x, xv[j].y * r * gv[j].y);
      yr[i] = o;
      xv[j] = __bfloat1622float2(o);
      amax = fmaxf(amax, fmaxf(fabsf(xv[j].x), fabsf(xv[j].y)));
    }
  }
  amax = block_max_rows(amax, s_part);
  float scale, inv_s;
  f16_row_scale(amax, scale, inv_s);
  if (threadIdx.x == 0) inv[m] = inv_s;
#pragma unroll
  for (int j = 0; j < kNormPairs; ++j) {
    const int i = threadIdx.x + j * kRowThreads;
    if (i < np) hr[i] = __floats2half2_rn(xv[j].x * scale, xv[j].y * scale);
  }
}

// Eq. 9 for a row held in registers as pairs: the per-token step from the maximum of the smoothed values, then the codes.
// v: the thread's smoothed values (pair j = elements 2 (thread + j * kRowThreads), +1); np pairs in the row.
template <int PAIRS>
__device__ __forceinline__ void quantize_row_pairs(const float2 (&v)[PAIRS], int np, float* s_part, int8_t* xq_row, float* dx_out) {
  float amax = 0.f;
#pragma unroll
  for (int j = 0; j < PAIRS; ++j)
    if ((int)threadIdx.x + j * kRowThreads < np) amax = fmaxf(amax, fmaxf(fabsf(v[j].x), fabsf(v[j].y)));
  amax = block_max_rows(amax, s_part);
  const float d = (amax == 0.f) ? 1.0f : __fdiv_rn(amax, 127.0f);
  if (threadIdx.x == 0) *dx_out = d;
#pragma unroll
  for (int j = 0; j < PAIRS; ++j) {
    const int i = (int)threadIdx.x + j * kRowThreads;
    if (i < np) {
      const int q0 = max(-127, min(127, __float2int_rn(__fdiv_rn(v[j].x, d))));
      const int q1 = max(-127, min(127, __float2int_rn(__fdiv_rn(v[j].y, d))));
      reinterpret_cast<char2*>(xq_row)[i] = make_char2((signed char)q0, (signed char)q1);
    }
  }
}

// RMSNorm whose output row is also smoothed and quantised per token for the W8A8 linear layer that follows.
__global__ void __launch_bounds__(kRowThreads)
rmsnorm_q8_kernel(const __nv_bfloat16* __restrict__ x, const __nv_bfloat16* __restrict__ g, const float* __restrict__ smooth, int H,
                  float eps, __nv_bfloat16* __restrict__ y, int8_t* __restrict__ xq, float* __restrict__ dx) {
  const int m = blockIdx.x;
  const __nv_bfloat162* xr = reinterpret_cast<const __nv_bfloat162*>(x + (size_t)m * H);
  const __nv_bfloat162* gr = reinterpret_cast<const __nv_bfloat162*>(g);
  __nv_bfloat162* yr = reinterpret_cast<__nv_bfloat162*>(y + (size_t)m * H);
  __shared__ float s_part[kRowThreads / 32];
  const int np = H / 2;
  float2 xv[kNormPairs];
  float ss = 0.f;
#pragma unroll
  for (int j = 0; j < kNormPairs; ++j) {
    const int i = threadIdx.x + j * kRowThreads;
    xv[j] = make_float2(0.f, 0.f);
    if (i < np) {
      xv[j] = __bfloat1622float2(xr[i]);
      ss += xv[j].x * xv[j].x + xv[j].y * xv[j].y;
    }
  }
  ss = warp_sum(ss);
  if ((threadIdx.x & 31) == 0) s_part[threadIdx.x >> 5] = ss;
  __syncthreads();
  float tot = 0.f;
#pragma unroll
  for (int i = 0; i < kRowThreads / 32; ++i) tot += s_part[i];
  const float r = 1.0f / sqrtf(tot / (float)H + eps);
#pragma unroll
  for (int j = 0; j < kNormPairs; ++j) {
    const int i = threadIdx.x + j * kRowThreads;
    if (i < np) {
      const float2 gg = __bfloat1622float2(gr[i]);
      const __nv_bfloat162 o = __floats2bfloat162_rn(xv[j].x * r * gg.x, xv[j].y * r * gg.y);
      yr[i] = o;
      const float2 h = __bfloat1622float2(o);
      const float2 sv = smooth != nullptr ? *reinterpret_cast<const float2*>(smooth + 2 * i) : make_float2(1.f, 1.f);
      xv[j] = make_float2(__fmul_rn(h.x, sv.x), __fmul_rn(h.y, sv.y));
    }
  }
  quantize_row_pairs<kNormPairs>(xv, np, s_part, xq + (size_t)m * H, dx + m);
}

// ---- RoPE table: cos/sin(pos * theta^(-2i/D)) evaluated in fp64, stored as fp32 -------------
__global__ void rope_table_kernel(float2* table, int max_pos, int D, double theta) {
  const int half = D / 2;
  const int idx = blockIdx.x * blockDim.x + threadIdx.x;
  if (idx >= max_pos * half) return;
  const int pos = idx / half, i = idx % half;
  const double inv_freq = pow(theta, -2.0 * (double)i / (double)D);
  double s, c;
  sincos((double)pos * inv_freq, &s, &c);
  table[idx] = make_float2((float)c, (float)s);
}

// ---- QK-RMSNorm + RoPE + KV append: one warp per (row, head) --------------------------------
template <int D>
__global__ void __launch_bounds__(128)
rope_append_kernel(__nv_bfloat16* __restrict__ qkv, const __nv_bfloat16* __restrict__ q_norm,
                   const __nv_bfloat16* __restrict__ k_norm, const float2* __restrict__ rope_table,
                   const int32_t* __restrict__ seq_len, const int32_t* __restrict__ block_len, BlockInfo bi, int T_max,
                   int Hq, int Hkv, float eps, __nv_bfloat16* __restrict__ k_cache, __nv_bfloat16* __restrict__ v_cache,
                   int s_max, int n_items) {
  constexpr int kPairs = D / 64;  // rotation pairs (i, i + D/2) per lane
  const int item = blockIdx.x * (blockDim.x >> 5) + (threadIdx.x >> 5);
  if (item >= n_items) return;
  const int lane = threadIdx.x & 31;
  const int heads = Hq + 2 * Hkv;
  const int m = item / heads, head = item % heads;
  const int b = m / T_max, i = m % T_max;
  if (!bi.valid[b] || i >= block_len[b]) return;
  const int P = seq_len[b];
  __nv_bfloat16* src = qkv + (size_t)m * heads * D + (size_t)head * D;

  if (head >= Hq + Hkv) {  // v head: copy into the cache
    const int hk = head - Hq - Hkv;
    __nv_bfloat16* dst = v_cache + (((size_t)b * Hkv + hk) * s_max + (P + i)) * D;
    if (lane < D / 8) reinterpret_cast<uint4*>(dst)[lane] = reinterpret_cast<const uint4*>(src)[lane];
    return;
  }
  const bool is_q = head < Hq;
  const __nv_bfloat16* gain = is_q ? q_norm : k_norm;
  float lo[kPairs], hi[kPairs];
  float ss = 0.f;
#pragma unroll
  for (int p = 0; p < kPairs; ++p) {
    const int d = lane + 32 * p;
    lo[p] = __bfloat162float(src[d]);
    hi[p] = __bfloat162float(src[d + D / 2]);
    ss += lo[p] * lo[p] + hi[p] * hi[p];
  }
  if (gain != nullptr) {
    ss = warp_sum(ss);
    const float r = 1.0f / sqrtf(ss / (float)D + eps);
#pragma unroll
    for (int p = 0; p < kPairs; ++p) {
      const int d = lane + 32 * p;
      lo[p] = lo[p] * r * __bfloat162float(gain[d]);
      hi[p] = hi[p] * r * __bfloat162float(gain[d + D / 2]);
    }
  }
  const int pos = P + bi.depth[m];
  __nv_bfloat16* dst = is_q ? src : k_cache + (((size_t)b * Hkv + (head - Hq)) * s_max + (P + i)) * D;
#pragma unroll
  for (int p = 0; p < kPairs; ++p) {
    const int d = lane + 32 * p;
    const float2 cs = rope_table[(size_t)pos * (D / 2) + d];
    dst[d] = __float2bfloat16_rn(lo[p] * cs.x - hi[p] * cs.y);
    dst[d + D / 2] = __float2bfloat16_rn(hi[p] * cs.x + lo[p] * cs.y);
  }
}

// ---- SwiGLU: act = silu(gate) * up -----------------------------------------------------------
__global__ void swiglu_kernel(const __nv_bfloat16* __restrict__ gu, int F, __nv_bfloat16* __restrict__ act) {
  const int m = blockIdx.y;
  const int f2 = blockIdx.x * blockDim.x + threadIdx.x;  // pair index
  if (f2 >= F / 2) return;
  const float2 gt = __bfloat1622float2(reinterpret_cast<const __nv_bfloat162*>(gu + (size_t)m * 2 * F)[f2]);
  const float2 up = __bfloat1622float2(reinterpret_cast<const __nv_bfloat162*>(gu + (size_t)m * 2 * F + F)[f2]);
  const float a0 = gt.x / (1.0f + expf(-gt.x)) * up.x;
  const float a1 = gt.y / (1.0f + expf(-gt.y)) * up.y;
  reinterpret_cast<__nv_bfloat162*>(act + (size_t)m * F)[f2] = __floats2bfloat162_rn(a0, a1);
}

// the same, one thread block per row, leaving the fp16 form of the row as well (the row stays in registers between
// the two passes: at most kActPairs pairs per thread, i.e. rows of up to 24576 elements)
constexpr int kActPairs = 12;

__global__ void __launch_bounds__(kRowThreads)
swiglu_f16_kernel(const __nv_bfloat16* __restrict__ gu, int F, __nv_bfloat16* __restrict__ act, __half* __restrict__ act16,
                  float* __restrict__ inv) {
  const int m = blockIdx.x;
  const __nv_bfloat162* gr = reinterpret_cast<const __nv_bfloat162*>(gu + (size_t)m * 2 * F);
  const __nv_bfloat162* ur = reinterpret_cast<const __nv_bfloat162*>(gu + (size_t)m * 2 * F + F);
  __nv_bfloat162* ar = reinterpret_cast<__nv_bfloat162*>(act + (size_t)m * F);
  __half2* hr = reinterpret_cast<__half2*>(act16 + (size_t)m * F);
  __shared__ float s_part[kRowThreads / 32];
  const int np = F / 2;
  __nv_bfloat162 av[kActPairs];
  float amax = 0.f;
#pragma unroll
  for (int j = 0; j < kActPairs; ++j) {
    const int i = threadIdx.x + j * kRowThreads;
    if (i < np) {
      const float2 gt = __bfloat1622float2(gr[i]);
      const float2 up = __bfloat1622float2(ur[i]);
      const float a0 = gt.x / (1.0f + expf(-gt.x)) * up.x;
      const float a1 = gt.y / (1.0f + expf(-gt.y)) * up.y;
      av[j] = __floats2bfloat162_rn(a0, a1);
      ar[i] = av[j];
      const float2 of = __bfloat1622float2(av[j]);
      amax = fmaxf(amax, fmaxf(fabsf(of.x), fabsf(of.y)));
    }
  }
  amax = block_max_rows(amax, s_part);
  float scale, inv_s;
  f16_row_scale(amax, scale, inv_s);
  if (threadIdx.x == 0) inv[m] = inv_s;
#pragma unroll
  for (int j = 0; j < kActPairs; ++j) {
    const int i = threadIdx.x + j * kRowThreads;
    if (i < np) {
      const float2 of = __bfloat1622float2(av[j]);
      hr[i] = __floats2half2_rn(of.x * scale, of.y * scale);
    }
  }
}

// SwiGLU whose output row is also smoothed and quantised per token for the W8A8 down projection.
__global__ void __launch_bounds__(kRowThreads)
swiglu_q8_kernel(const __nv_bfloat16* __restrict__ gu, const float* __restrict__ smooth, int F, __nv_bfloat16* __restrict__ act,
                 int8_t* __restrict__ xq, float* __restrict__ dx) {
  const int m = blockIdx.x;
  const __nv_bfloat162* gr = reinterpret_cast<const __nv_bfloat162*>(gu + (size_t)m * 2 * F);
  const __nv_bfloat162* ur = reinterpret_cast<const __nv_bfloat162*>(gu + (size_t)m * 2 * F + F);
  __nv_bfloat162* ar = reinterpret_cast<__nv_bfloat162*>(act + (size_t)m * F);
  __shared__ float s_part[kRowThreads / 32];
  const int np = F / 2;
  float2 v[kActPairs];
#pragma unroll
  for (int j = 0; j < kActPairs; ++j) {
    const int i = threadIdx.x + j * kRowThreads;
    v[j] = make_float2(0.f, 0.f);
    if (i < np) {
      const float2 gt = __bfloat1622float2(gr[i]);
      const float2 up = __bfloat1622float2(ur[i]);
      const __nv_bfloat162 o = __floats2bfloat162_rn(gt.x / (1.0f + expf(-gt.x)) * up.x, gt.y / (1.0f + expf(-gt.y)) * up.y);
      ar[i] = o;
      const float2 h = __bfloat1622float2(o);
      const float2 sv = smooth != nullptr ? *reinterpret_cast<const float2*>(smooth + 2 * i) : make_float2(1.f, 1.f);
      v[j] = make_float2(__fmul_rn(h.x, sv.x), __fmul_rn(h.y, sv.y));
    }
  }
  quantize_row_pairs<kActPairs>(v, np, s_part, xq + (size_t)m * F, dx + m);
}

// ---- arg-max over the vocabulary, lowest index on ties ---------------------------------------
// A row is cut into segments, one thread block each; a block's best (value, index) goes into the row's 64-bit key
// by atomicMax: the value's bits made order-preserving in the high word, the complemented index in the low word,
// so the largest key is the largest value and, among equals, the lowest index.  NaNs never enter; a row without
// any number keeps key 0 and decodes to index 0.
constexpr int kArgmaxSeg = 8192;

__device__ __forceinline__ unsigned long long argmax_key(float x, int idx) {
  x += 0.0f;                                            // -0 -> +0: they compare equal
  uint32_t u = __float_as_uint(x);
  u = (u & 0x80000000u) ? ~u : (u | 0x80000000u);
  return ((unsigned long long)u << 32) | (unsigned long long)(0xffffffffu - (uint32_t)idx);
}

__global__ void __launch_bounds__(256) argmax_segment_kernel(const float* __restrict__ logits, int V, unsigned long long* keys) {
  const int m = blockIdx.y;
  const float* row = logits + (size_t)m * V;
  const int v0 = blockIdx.x * kArgmaxSeg;
  const int v1 = min(V, v0 + kArgmaxSeg);
  unsigned long long best = 0ull;
  if ((V & 3) == 0) {
    for (int v = v0 + threadIdx.x * 4; v < v1; v += 256 * 4) {
      const float4 f = *reinterpret_cast<const float4*>(row + v);
      const float e[4] = {f.x, f.y, f.z, f.w};
#pragma unroll
      for (int j = 0; j < 4; ++j)
        if (e[j] == e[j]) {
          const unsigned long long k = argmax_key(e[j], v + j);
          best = k > best ? k : best;
        }
    }
  } else {
    for (int v = v0 + threadIdx.x; v < v1; v += 256) {
      const float x = row[v];
      if (x == x) {
        const unsigned long long k = argmax_key(x, v);
        best = k > best ? k : best;
      }
    }
  }
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) {
    const unsigned long long ob = __shfl_xor_sync(0xffffffffu, best, o);
    best = ob > best ? ob : best;
  }
  if ((threadIdx.x & 31) == 0 && best != 0ull) atomicMax(keys + m, best);
}

__global__ void argmax_decode_kernel(const unsigned long long* __restrict__ keys, int M, int32_t* top1) {
  const int m = blockIdx.x * blockDim.x + threadIdx.x;
  if (m >= M) return;
  const unsigned long long k = keys[m];
  top1[m] = k == 0ull ? 0 : (int32_t)(0xffffffffu - (uint32_t)(k & 0xffffffffull));
}

// ---- greedy acceptance: one thread per sequence ----------------------------------------------
__global__ void accept_kernel(const int32_t* __restrict__ tokens, const int32_t* __restrict__ parents,
                              const int32_t* __restrict__ block_len, const int32_t* __restrict__ top1, BlockInfo bi,
                              int B, int T_max, int32_t* accept_len, int32_t* bonus, int32_t* accept_path) {
  const int b = blockIdx.x * blockDim.x + threadIdx.x;
  if (b >= B) return;
  const int base = b * T_max;
  if (!bi.valid[b]) {   // a skipped sequence: -1 tells quasar_kv_commit to leave its cache and seq_len alone
    accept_len[b] = -1;
    bonus[b] = -1;
    if (accept_path) for (int d = 0; d < T_max; ++d) accept_path[base + d] = -1;
    return;
  }
  const int T = block_len[b];
  int cur = 0, n = 0;
  if (accept_path) accept_path[base] = 0;
  while (true) {
    int nxt = -1;
    const int want = top1[base + cur];
    for (int c = cur + 1; c < T; ++c) {
      const int p = parents ? parents[base + c] : c - 1;
      if (p == cur && tokens[base + c] == want) { nxt = c; break; }
    }
    if (nxt < 0) break;
    cur = nxt;
    ++n;
    if (accept_path) accept_path[base + n] = cur;
  }
  accept_len[b] = n;
  bonus[b] = top1[base + cur];
  if (accept_path) for (int d = n + 1; d < T_max; ++d) accept_path[base + d] = -1;
}

// ---- commit: (tree) move accepted rows into place, then bump seq_len --------------------------
// One thread per 16-byte piece of a (layer, sequence, kv head) row; depths are walked in
// increasing order inside the thread, which keeps every source slot intact until it is read
// (the accepted row at depth d has block index >= d).
__global__ void kv_gather_kernel(__nv_bfloat16* __restrict__ k_cache, __nv_bfloat16* __restrict__ v_cache,
                                 const int32_t* __restrict__ seq_len, const int32_t* __restrict__ accept_len,
                                 const int32_t* __restrict__ accept_path, int L, int B_cache, int B, int T_max,
                                 int Hkv, int D, int s_max) {
  const int chunks = D / 8;
  const size_t total = (size_t)L * B * Hkv * chunks;
  const size_t idx = (size_t)blockIdx.x * blockDim.x + threadIdx.x;
  if (idx >= total) return;
  const int c = (int)(idx % chunks);
  size_t r = idx / chunks;
  const int hk = (int)(r % Hkv); r /= Hkv;
  const int b = (int)(r % B);
  const int l = (int)(r / B);
  const int n = accept_len[b];
  const int P = seq_len[b];
  if (n < 0 || n >= T_max || P < 0) return;
  const size_t base = (((size_t)l * B_cache + b) * Hkv + hk) * (size_t)s_max;
  for (int d = 1; d <= n; ++d) {
    const int j = accept_path[b * T_max + d];
    if (j == d || j < d || j >= T_max || P + j >= s_max) continue;
    uint4* kd = reinterpret_cast<uint4*>(k_cache + (base + P + d) * D) + c;
    uint4* vd = reinterpret_cast<uint4*>(v_cache + (base + P + d) * D) + c;
    *kd = *(reinterpret_cast<const uint4*>(k_cache + (base + P + j) * D) + c);
    *vd = *(reinterpret_cast<const uint4*>(v_cache + (base + P + j) * D) + c);
  }
}

__global__ void seq_bump_kernel(int32_t* seq_len, const int32_t* __restrict__ accept_len, int B, int T_max, int s_max) {
  const int b = blockIdx.x * blockDim.x + threadIdx.x;
  if (b >= B) return;
  const int n = accept_len[b];
  if (n < 0 || n >= T_max) return;
  const int v = seq_len[b] + 1 + n;
  if (v <= s_max) seq_len[b] = v;
}

}  // namespace

int launch_block_prep(const int32_t* tokens, const int32_t* parents, const int32_t* block_len, const int32_t* seq_len,
                      int B, int T_max, int s_max, int vocab, BlockInfo bi, int32_t* status, cudaStream_t stream) {
  block_prep_kernel<<<(B + 63) / 64, 64, 0, stream>>>(tokens, parents, block_len, seq_len, B, T_max, s_max, vocab, bi,
                                                     status);
  QUASAR_LAUNCH_CHECK();
  return QUASAR_OK;
}

int launch_embed(const int32_t* tokens, const __nv_bfloat16* embed, int M, int H, int vocab, __nv_bfloat16* x,
                 cudaStream_t stream) {
  embed_kernel<<<M, 128, 0, stream>>>(tokens, embed, H, vocab, x);
  QUASAR_LAUNCH_CHECK();
  return QUASAR_OK;
}

int launch_rmsnorm(const __nv_bfloat16* x, const __nv_bfloat16* g, int M, int H, float eps, __nv_bfloat16* y,
                   cudaStream_t stream) {
  rmsnorm_kernel<<<M, 256, 0, stream>>>(x, g, H, eps, y);
  QUASAR_LAUNCH_CHECK();
  return QUASAR_OK;
}

int launch_rmsnorm_f16(const __nv_bfloat16* x, const __nv_bfloat16* g, int M, int H, float eps, __nv_bfloat16* y, void* y16,
                       float* inv, cudaStream_t stream) {
  if (H > 2 * kNormPairs * kRowThreads) { set_error("rmsnorm_f16: rows of %d elements (at most %d)", H, 2 * kNormPairs * kRowThreads); return QUASAR_ERR_SHAPE; }
  rmsnorm_f16_kernel<false><<<M, kRowThreads, 0, stream>>>(nullptr, 0, 0, nullptr, nullptr, const_cast<__nv_bfloat16*>(x), g, H, eps, y,
                                                    reinterpret_cast<__half*>(y16), inv);
  QUASAR_LAUNCH_CHECK();
  return QUASAR_OK;
}

int launch_reduce_residual_rmsnorm_f16(const float* partial, int nsplit, int mpad, const float* dx, const float* dw,
                                       __nv_bfloat16* x, const __nv_bfloat16* g, int M, int H, float eps, __nv_bfloat16* y,
                                       void* y16, float* inv, cudaStream_t stream) {
  if (H > 2 * kNormPairs * kRowThreads) { set_error("rmsnorm_f16: rows of %d elements (at most %d)", H, 2 * kNormPairs * kRowThreads); return QUASAR_ERR_SHAPE; }
  rmsnorm_f16_kernel<true><<<M, kRowThreads, 0, stream>>>(partial, nsplit, mpad, dx, dw, x, g, H, eps, y, reinterpret_cast<__half*>(y16),
                                                   inv);
  QUASAR_LAUNCH_CHECK();
  return QUASAR_OK;
}

int launch_rmsnorm_q8(const __nv_bfloat16* x, const __nv_bfloat16* g, const float* smooth, int M, int H, float eps,
                      __nv_bfloat16* y, int8_t* xq, float* dx, cudaStream_t stream) {
  if (H > 2 * kNormPairs * kRowThreads) { set_error("rmsnorm_q8: rows of %d elements (at most %d)", H, 2 * kNormPairs * kRowThreads); return QUASAR_ERR_SHAPE; }
  rmsnorm_q8_kernel<<<M, kRowThreads, 0, stream>>>(x, g, smooth, H, eps, y, xq, dx);
  QUASAR_LAUNCH_CHECK();
  return QUASAR_OK;
}

int launch_swiglu_q8(const __nv_bfloat16* gu, const float* smooth, int M, int F, __nv_bfloat16* act, int8_t* xq, float* dx,
                     cudaStream_t stream) {
  if (F > 2 * kActPairs * kRowThreads) { set_error("swiglu_q8: rows of %d elements (at most %d)", F, 2 * kActPairs * kRowThreads); return QUASAR_ERR_SHAPE; }
  swiglu_q8_kernel<<<M, kRowThreads, 0, stream>>>(gu, smooth, F, act, xq, dx);
  QUASAR_LAUNCH_CHECK();
  return QUASAR_OK;
}

int launch_swiglu_f16(const __nv_bfloat16* gu, int M, int F, __nv_bfloat16* act, void* act16, float* inv, cudaStream_t stream) {
  if (F > 2 * kActPairs * kRowThreads) { set_error("swiglu_f16: rows of %d elements (at most %d)", F, 2 * kActPairs * kRowThreads); return QUASAR_ERR_SHAPE; }
  swiglu_f16_kernel<<<M, kRowThreads, 0, stream>>>(gu, F, act, reinterpret_cast<__half*>(act16), inv);
  QUASAR_LAUNCH_CHECK();
  return QUASAR_OK;
}

int launch_rope_table(float2* table, int max_pos, int D, float theta, cudaStream_t stream) {
  const int total = max_pos * (D / 2);
  rope_table_kernel<<<(total + 255) / 256, 256, 0, stream>>>(table, max_pos, D, (double)theta);
  QUASAR_LAUNCH_CHECK();
  return QUASAR_OK;
}

int launch_rope_append(__nv_bfloat16* qkv, const __nv_bfloat16* q_norm, const __nv_bfloat16* k_norm,
                       const float2* rope_table, const int32_t* seq_len, const int32_t* block_len, BlockInfo bi, int B,
                       int T_max, int Hq, int Hkv, int D, float eps, __nv_bfloat16* k_cache_layer,
                       __nv_bfloat16* v_cache_layer, int s_max, cudaStream_t stream) {
  const int n_items = B * T_max * (Hq + 2 * Hkv);
  const int grid = (n_items + 3) / 4;
  if (D == 128) {
    rope_append_kernel<128><<<grid, 128, 0, stream>>>(qkv, q_norm, k_norm, rope_table, seq_len, block_len, bi, T_max,
                                                       Hq, Hkv, eps, k_cache_layer, v_cache_layer, s_max, n_items);
  } else if (D == 64) {
    rope_append_kernel<64><<<grid, 128, 0, stream>>>(qkv, q_norm, k_norm, rope_table, seq_len, block_len, bi, T_max,
                                                      Hq, Hkv, eps, k_cache_layer, v_cache_layer, s_max, n_items);
  } else {
    set_error("head_dim %d not supported (64 or 128)", D);
    return QUASAR_ERR_SHAPE;
  }
  QUASAR_LAUNCH_CHECK();
  return QUASAR_OK;
}

int launch_swiglu(const __nv_bfloat16* gu, int M, int F, __nv_bfloat16* act, cudaStream_t stream) {
  dim3 grid((F / 2 + 255) / 256, M);
  swiglu_kernel<<<grid, 256, 0, stream>>>(gu, F, act);
  QUASAR_LAUNCH_CHECK();
  return QUASAR_OK;
}

int launch_argmax(const float* logits, int M, int V, int32_t* top1, unsigned long long* keys, cudaStream_t stream) {
  QUASAR_CUDA_CHECK(cudaMemsetAsync(keys, 0, (size_t)M * sizeof(unsigned long long), stream));
  argmax_segment_kernel<<<dim3((V + kArgmaxSeg - 1) / kArgmaxSeg, M), 256, 0, stream>>>(logits, V, keys);
  QUASAR_LAUNCH_CHECK();
  argmax_decode_kernel<<<(M + 127) / 128, 128, 0, stream>>>(keys, M, top1);
  QUASAR_LAUNCH_CHECK();
  return QUASAR_OK;
}

int launch_accept(const int32_t* tokens, const int32_t* parents, const int32_t* block_len, const int32_t* top1,
                  BlockInfo bi, int B, int T_max, int32_t* accept_len, int32_t* bonus, int32_t* accept_path,
                  cudaStream_t stream) {
  accept_kernel<<<(B + 63) / 64, 64, 0, stream>>>(tokens, parents, block_len, top1, bi, B, T_max, accept_len, bonus,
                                                 accept_path);
  QUASAR_LAUNCH_CHECK();
  return QUASAR_OK;
}

int launch_kv_commit(__nv_bfloat16* k_cache, __nv_bfloat16* v_cache, int32_t* seq_len, const int32_t* accept_len,
                     const int32_t* accept_path, int L, int B_cache, int B, int T_max, int Hkv, int D, int s_max,
                     cudaStream_t stream) {
  if (accept_path != nullptr) {
    const size_t total = (size_t)L * B * Hkv * (D / 8);
    kv_gather_kernel<<<(unsigned)((total + 255) / 256), 256, 0, stream>>>(k_cache, v_cache, seq_len, accept_len,
                                                                          accept_path, L, B_cache, B, T_max, Hkv, D,
                                                                          s_max);
    QUASAR_LAUNCH_CHECK();
  }
  seq_bump_kernel<<<(B + 63) / 64, 64, 0, stream>>>(seq_len, accept_len, B, T_max, s_max);
  QUASAR_LAUNCH_CHECK();
  return QUASAR_OK;
}

}  // namespace quasar
