// C ABI of the library: argument checks, the model object, and the sequence of launches
// that makes up one verification pass (Section 3.1 "Verification", Section 3.3).
#include <math.h>
#include <stdarg.h>
#include <stdio.h>
#include <string.h>

#include <algorithm>
#include <atomic>
#include <new>
#include <vector>

#include "common.cuh"
#include "megakernel.cuh"

namespace quasar {

static thread_local char g_err[512] = "";
static std::atomic<long long> g_launches{0};

void set_error(const char* fmt, ...) {
  va_list ap;
  va_start(ap, fmt);
  vsnprintf(g_err, sizeof(g_err), fmt, ap);
  va_end(ap);
}

void count_launch(int n) { g_launches.fetch_add(n, std::memory_order_relaxed); }

}  // namespace quasar

using namespace quasar;

struct quasar_model {
  quasar_config cfg;
  std::vector<quasar_layer_weights> layers;
  quasar_weights w;
  float2* rope_table = nullptr;
  void* trace_buf = nullptr;
  size_t trace_bytes = 0;
  // persistent single-kernel path
  MegaJob* mega_jobs = nullptr;     // device
  MegaLayer* mega_layers = nullptr; // device
  unsigned char* mega_weights = nullptr;  // device: every matrix again, permuted for the persistent kernel
  int mega_ncta = 0;                // 0: not available on this device
  int path = 0;                     // 0 auto, 1 one kernel per step, 2 persistent kernel
  unsigned long long wait_budget_ns = 2000000000ull;   // bound of every device-side wait of the persistent kernel
  unsigned barrier_extra = 0;       // test of the failure path only (quasar_set_wait_budget)
};

struct quasar_plan {
  cudaGraph_t graph = nullptr;
  cudaGraphExec_t exec = nullptr;   // null: the pass is a single persistent kernel, launched directly
  quasar_model* model = nullptr;
  quasar_kv kv;
  float* logits_out = nullptr;
  void* workspace = nullptr;
  size_t workspace_bytes = 0;
  const int32_t *tokens, *parents, *block_len;
  int32_t *accept_len, *bonus, *accept_path, *status;
  int B, T_max;
  int kernels = 0;  // kernel nodes one replay runs
};

namespace {

size_t align_up(size_t v, size_t a = 256) { return (v + a - 1) / a * a; }

// Layout of the verify workspace; every offset is a multiple of 256 bytes.
struct Workspace {
  size_t x, h, qkv, attn, gu, act, attn16, act16, h16, inv3, keys, logits, top1, anc, depth, valid, lin, att, cand, ss_part, amax, attn_count, barrier, total;
  size_t lin_bytes, att_bytes;
};

constexpr int kMaxGrid = 1024;  // upper bound on CTAs of the persistent kernel (SM count)

Workspace layout(const quasar_config& c, int B, int T_max, int s_max) {
  Workspace w;
  const size_t M = (size_t)B * T_max;
  const size_t qkv_w = (size_t)(c.n_q_heads + 2 * c.n_kv_heads) * c.head_dim;
  size_t off = 0;
  auto take = [&](size_t bytes) { size_t o = off; off += align_up(bytes); return o; };
  w.x = take(M * c.hidden * 2);
  w.h = take(M * c.hidden * 2);
  w.qkv = take(M * qkv_w * 2);
  w.attn = take(M * (size_t)c.n_q_heads * c.head_dim * 2);
  w.gu = take(M * 2 * (size_t)c.ffn * 2);
  w.act = take(M * (size_t)c.ffn * 2);
  w.attn16 = take(M * (size_t)c.n_q_heads * c.head_dim * 2);
  w.act16 = take(M * (size_t)c.ffn * 2);
  w.h16 = take(M * (size_t)c.hidden * 2);
  w.inv3 = take(3 * align_up(M * 4));
  w.keys = take(M * 8);
  w.logits = take(M * (size_t)c.vocab * 4);
  w.top1 = take(M * 4);
  w.anc = take(M * 8);
  w.depth = take(M * 4);
  w.valid = take((size_t)B * 4);
  size_t lin = 0;
  const int64_t shapes[5][2] = {{(int64_t)qkv_w, c.hidden},
                                {c.hidden, (int64_t)c.n_q_heads * c.head_dim},
                                {2 * (int64_t)c.ffn, c.hidden},
                                {c.hidden, c.ffn},
                                {c.vocab, c.hidden}};
  for (auto& s : shapes) {
    size_t b = linear_workspace_bytes((int64_t)M, s[0], s[1]);
    if (c.act_dtype == QUASAR_A_INT8) {
      const size_t b8 = linear_w8a8_workspace_bytes((int64_t)M, s[0], s[1]);
      b = b8 > b ? b8 : b;
    }
    lin = b > lin ? b : lin;
  }
  w.lin_bytes = lin;
  w.lin = take(lin);
  w.att_bytes = attention_workspace_bytes(B, T_max, c.n_q_heads, c.n_kv_heads, c.head_dim, s_max);
  {
    const size_t rows = (size_t)B * c.n_kv_heads * mega_attn_nchunk(s_max) * mega_attn_rpad(T_max, c.n_q_heads, c.n_kv_heads);
    const size_t mega = rows * c.head_dim * sizeof(float) + rows * 2 * sizeof(float);
    if (mega > w.att_bytes) w.att_bytes = mega;
  }
  w.att = take(w.att_bytes);
  w.cand = take((size_t)kMaxGrid * 8 * 2 * sizeof(float));
  w.ss_part = take((size_t)kMaxGrid * 8 * sizeof(float));
  w.amax = take((size_t)(4 * c.n_layers + 1) * 8 * sizeof(unsigned));
  w.attn_count = take((size_t)(c.n_layers > 0 ? c.n_layers : 1) * B * c.n_kv_heads * sizeof(unsigned));
  w.barrier = take(256);
  w.total = off;
  return w;
}

int check_cfg(const quasar_config& c) {
  if (c.n_layers < 0 || c.hidden <= 0 || c.n_q_heads <= 0 || c.n_kv_heads <= 0 || c.ffn <= 0 || c.vocab <= 0 ||
      c.max_seq <= 0) {
    set_error("config: non-positive size");
    return QUASAR_ERR_INVALID_ARG;
  }
  if (c.weight_dtype != QUASAR_W_INT8 && c.weight_dtype != QUASAR_W_BF16) {
    set_error("config: weight_dtype %d", c.weight_dtype);
    return QUASAR_ERR_INVALID_ARG;
  }
  if (c.weights_in_place && c.act_dtype != QUASAR_A_BF16) {
    set_error("config: weights_in_place needs the persistent kernel, which handles bf16 activations only");
    return QUASAR_ERR_INVALID_ARG;
  }
  if (c.act_dtype != QUASAR_A_BF16 && !(c.act_dtype == QUASAR_A_INT8 && c.weight_dtype == QUASAR_W_INT8)) {
    set_error("config: act_dtype %d (int8 activations need int8 weights)", c.act_dtype);
    return QUASAR_ERR_INVALID_ARG;
  }
  if ((c.head_dim != 64 && c.head_dim != 128) || c.hidden % 16 || c.ffn % 16 || c.n_q_heads % c.n_kv_heads ||
      c.n_q_heads / c.n_kv_heads > 8 || ((int64_t)c.n_q_heads * c.head_dim) % 16) {
    set_error("config: unsupported shape (head_dim 64/128, hidden and ffn multiples of 16, group size <= 8)");
    return QUASAR_ERR_SHAPE;
  }
  return QUASAR_OK;
}

#define REQUIRE_PTR(p, name)                                  \
  do {                                                        \
    if ((p) == nullptr) {                                     \
      set_error("%s is NULL", name);                          \
      return QUASAR_ERR_INVALID_ARG;                          \
    }                                                         \
    if (!aligned16(p)) {                                      \
      set_error("%s is not 16-byte aligned", name);           \
      return QUASAR_ERR_ALIGN;                                \
    }                                                         \
  } while (0)

struct TraceCursor {
  unsigned char* base;
  size_t off, cap;
  cudaStream_t stream;
  int put(const void* src, size_t bytes) {
    if (base == nullptr) return QUASAR_OK;
    if (off + bytes > cap) {
      set_error("trace buffer too small");
      return QUASAR_ERR_CAPACITY;
    }
    QUASAR_CUDA_CHECK(cudaMemcpyAsync(base + off, src, bytes, cudaMemcpyDeviceToDevice, stream));
    off += bytes;
    return QUASAR_OK;
  }
};

#define TRY(expr)                       \
  do {                                  \
    int rc__ = (expr);                  \
    if (rc__ != QUASAR_OK) return rc__; \
  } while (0)

bool uses_persistent_kernel(const quasar_model* m, int B, int T_max) {
  const quasar_config& c = m->cfg;
  return m->path != 1 && m->mega_ncta > 0 && m->mega_ncta <= kMaxGrid && m->trace_buf == nullptr &&
         mega_supported(B * T_max, T_max, c.n_q_heads, c.n_kv_heads, c.head_dim);
}

int verify_impl(quasar_model* m, const quasar_kv* kv, const int32_t* tokens, const int32_t* parents,
                const int32_t* block_len, int32_t B, int32_t T_max, float* logits_out, int32_t* accept_len,
                int32_t* bonus, int32_t* accept_path, void* workspace, size_t workspace_bytes, int32_t* status,
                cudaStream_t stream) {
  if (m == nullptr || kv == nullptr) {
    set_error("model or kv is NULL");
    return QUASAR_ERR_INVALID_ARG;
  }
  const quasar_config& c = m->cfg;
  if (B < 1 || T_max < 1 || T_max > QUASAR_MAX_BLOCK) {
    set_error("verify: B=%d T_max=%d (T_max must be 1..%d)", B, T_max, QUASAR_MAX_BLOCK);
    return QUASAR_ERR_SHAPE;
  }
  if (B > kv->batch || kv->s_max > c.max_seq || kv->s_max < 1) {
    set_error("verify: batch %d exceeds cache batch %d, or s_max %d outside 1..max_seq %d", B, kv->batch, kv->s_max,
              c.max_seq);
    return QUASAR_ERR_CAPACITY;
  }
  REQUIRE_PTR(kv->k, "kv.k");
  REQUIRE_PTR(kv->v, "kv.v");
  REQUIRE_PTR(kv->seq_len, "kv.seq_len");
  REQUIRE_PTR(tokens, "tokens");
  REQUIRE_PTR(block_len, "block_len");
  REQUIRE_PTR(accept_len, "accept_len");
  REQUIRE_PTR(bonus, "bonus");
  REQUIRE_PTR(workspace, "workspace");
  REQUIRE_PTR(status, "status");
  if (parents && !aligned16(parents)) { set_error("parents is not 16-byte aligned"); return QUASAR_ERR_ALIGN; }
  if (logits_out && !aligned16(logits_out)) { set_error("logits_out is not 16-byte aligned"); return QUASAR_ERR_ALIGN; }
  if (accept_path && !aligned16(accept_path)) { set_error("accept_path is not 16-byte aligned"); return QUASAR_ERR_ALIGN; }
  const Workspace ws = layout(c, B, T_max, kv->s_max);
  if (workspace_bytes < ws.total) {
    set_error("verify: workspace of %zu bytes, need %zu", workspace_bytes, ws.total);
    return QUASAR_ERR_CAPACITY;
  }

  unsigned char* wsp = reinterpret_cast<unsigned char*>(workspace);
  __nv_bfloat16* x = reinterpret_cast<__nv_bfloat16*>(wsp + ws.x);
  __nv_bfloat16* h = reinterpret_cast<__nv_bfloat16*>(wsp + ws.h);
  __nv_bfloat16* qkv = reinterpret_cast<__nv_bfloat16*>(wsp + ws.qkv);
  __nv_bfloat16* attn = reinterpret_cast<__nv_bfloat16*>(wsp + ws.attn);
  __nv_bfloat16* gu = reinterpret_cast<__nv_bfloat16*>(wsp + ws.gu);
  __nv_bfloat16* act = reinterpret_cast<__nv_bfloat16*>(wsp + ws.act);
  float* logits = logits_out ? logits_out : reinterpret_cast<float*>(wsp + ws.logits);
  int32_t* top1 = reinterpret_cast<int32_t*>(wsp + ws.top1);
  BlockInfo bi;
  bi.anc = reinterpret_cast<uint64_t*>(wsp + ws.anc);
  bi.depth = reinterpret_cast<int32_t*>(wsp + ws.depth);
  bi.valid = reinterpret_cast<int32_t*>(wsp + ws.valid);
  void* lin = wsp + ws.lin;
  void* att = wsp + ws.att;

  const int M = B * T_max;
  const int H = c.hidden, D = c.head_dim, Hq = c.n_q_heads, Hkv = c.n_kv_heads, F = c.ffn;
  const int qkv_w = (Hq + 2 * Hkv) * D;
  const int wd = c.weight_dtype;
  const bool a8 = c.act_dtype == QUASAR_A_INT8;
  // one linear layer of the pass: weight-only (Eq. 8 with bf16 activations) or the paper's W8A8 form (Eq. 9-10)
  auto linear = [&](const __nv_bfloat16* in, const void* w, const float* delta, const float* smooth, int64_t N, int64_t K,
                    void* out, bool out_f32, const __nv_bfloat16* res) -> int {
    if (a8)
      return launch_linear_w8a8(in, smooth, reinterpret_cast<const int8_t*>(w), delta, M, N, K, out, out_f32, res, nullptr,
                                lin, ws.lin_bytes, status, stream);
    return launch_linear(in, w, delta, wd, M, N, K, out, out_f32, res, lin, ws.lin_bytes, stream, status);
  };
  const size_t layer_stride = (size_t)kv->batch * Hkv * (size_t)kv->s_max * D;
  TraceCursor tr{reinterpret_cast<unsigned char*>(m->trace_buf), 0, m->trace_bytes, stream};

  const bool can_mega = m->mega_ncta > 0 && m->mega_ncta <= kMaxGrid && m->trace_buf == nullptr &&
                        mega_supported(M, T_max, Hq, Hkv, D);
  if (m->path == 2 && !can_mega) {
    set_error("verify: the persistent kernel handles at most 8 block rows in total and no trace");
    return QUASAR_ERR_SHAPE;
  }
  if (can_mega && m->path != 1) {
    MegaParams p;
    p.jobs = m->mega_jobs; p.layers = m->mega_layers; p.n_jobs = 4 * c.n_layers + 1; p.L = c.n_layers;
    p.B = B; p.T_max = T_max; p.M = M; p.H = H; p.Hq = Hq; p.Hkv = Hkv; p.vocab = c.vocab; p.s_max = kv->s_max;
    p.kv_batch = kv->batch; p.rms_eps = c.rms_eps;
    p.embed = reinterpret_cast<const __nv_bfloat16*>(m->w.embed);
    p.rope_table = m->rope_table;
    p.tokens = tokens; p.parents = parents; p.block_len = block_len; p.seq_len = kv->seq_len;
    p.k_cache = reinterpret_cast<__nv_bfloat16*>(kv->k); p.v_cache = reinterpret_cast<__nv_bfloat16*>(kv->v);
    p.x = x; p.qkv = qkv; p.attn = attn; p.act = act;
    p.attn16 = reinterpret_cast<unsigned short*>(wsp + ws.attn16);
    p.act16 = reinterpret_cast<unsigned short*>(wsp + ws.act16); p.logits = logits_out; p.top1 = top1; p.bi = bi;
    p.attn_nchunk = mega_attn_nchunk(kv->s_max);
    p.attn_rpad = mega_attn_rpad(T_max, Hq, Hkv);
    const size_t rows = (size_t)B * Hkv * p.attn_nchunk * p.attn_rpad;
    p.o_part = reinterpret_cast<float*>(att);
    p.ml_part = p.o_part + rows * D;
    p.cand_val = reinterpret_cast<float*>(wsp + ws.cand);
    p.cand_idx = reinterpret_cast<int*>(wsp + ws.cand + (size_t)kMaxGrid * 8 * sizeof(float));
    p.ss_part = reinterpret_cast<float*>(wsp + ws.ss_part);
    p.amax_buf = reinterpret_cast<unsigned*>(wsp + ws.amax);
    p.attn_count = reinterpret_cast<unsigned*>(wsp + ws.attn_count);
    p.barrier = reinterpret_cast<unsigned*>(wsp + ws.barrier);
    p.accept_len = accept_len; p.bonus = bonus; p.accept_path = accept_path; p.status = status;
    p.wait_budget_ns = m->wait_budget_ns; p.barrier_extra = m->barrier_extra;
    QUASAR_CUDA_CHECK(cudaMemsetAsync(p.barrier, 0, 256, stream));
    return launch_verify_mega(p, wd, D, m->mega_ncta, stream);
  }

  // arrival counters of the split-K reduction start at zero and reset themselves
  QUASAR_CUDA_CHECK(cudaMemsetAsync(lin, 0, ws.lin_bytes < 65536 ? ws.lin_bytes : 65536, stream));
  TRY(launch_block_prep(tokens, parents, block_len, kv->seq_len, B, T_max, kv->s_max, c.vocab, bi, status, stream));
  TRY(launch_embed(tokens, reinterpret_cast<const __nv_bfloat16*>(m->w.embed), M, H, c.vocab, x, stream));
  TRY(tr.put(x, (size_t)M * H * 2));

  // Blocks of 9..80 rows with int8 weights and 16-bit activations: every linear layer is the tcgen05 kernel, which
  // wants its operand as fp16 rows times a power of two.  The kernel that produces an operand writes that form too, and
  // the kernel after a residual linear layer adds up its k-ranges, so a layer is 12 launches instead of 17.
  bool fused = !a8 && wd == QUASAR_W_INT8 && M > 8 && M <= 80 && H <= 8192 && F <= 24576;   // (rows the fused row kernels hold in registers)
  {
    const int64_t shapes[5][2] = {{qkv_w, H}, {H, (int64_t)Hq * D}, {2 * (int64_t)F, H}, {H, F}, {c.vocab, H}};
    for (auto& sh : shapes) fused = fused && umma_w8a16_usable(M, sh[0], sh[1]);
  }
  if (fused) {
    void* h16 = wsp + ws.h16;
    void* attn16 = wsp + ws.attn16;
    void* act16 = wsp + ws.act16;
    float* inv_h = reinterpret_cast<float*>(wsp + ws.inv3);
    float* inv_a = reinterpret_cast<float*>(wsp + ws.inv3 + align_up((size_t)M * 4));
    float* inv_f = reinterpret_cast<float*>(wsp + ws.inv3 + 2 * align_up((size_t)M * 4));
    float* partial = reinterpret_cast<float*>(reinterpret_cast<unsigned char*>(lin) + 65536);
    auto norm_of = [&](int l) {
      return reinterpret_cast<const __nv_bfloat16*>(l < c.n_layers ? m->layers[l].attn_norm : m->w.final_norm);
    };
    TRY(launch_rmsnorm_f16(x, norm_of(0), M, H, c.rms_eps, h, h16, inv_h, stream));
    for (int l = 0; l < c.n_layers; ++l) {
      const quasar_layer_weights& L = m->layers[l];
      __nv_bfloat16* kc = reinterpret_cast<__nv_bfloat16*>(kv->k) + (size_t)l * layer_stride;
      __nv_bfloat16* vc = reinterpret_cast<__nv_bfloat16*>(kv->v) + (size_t)l * layer_stride;
      int ns = 1, mpad = 16;
      TRY(tr.put(h, (size_t)M * H * 2));
      TRY(launch_umma_w8a16_prepared(h16, inv_h, reinterpret_cast<const int8_t*>(L.qkv_w), L.qkv_delta, M, qkv_w, H, qkv, false,
                                     nullptr, partial, true, status, stream));
      TRY(tr.put(qkv, (size_t)M * qkv_w * 2));
      TRY(launch_rope_append(qkv, reinterpret_cast<const __nv_bfloat16*>(c.qk_norm ? L.q_norm : nullptr),
                             reinterpret_cast<const __nv_bfloat16*>(c.qk_norm ? L.k_norm : nullptr), m->rope_table,
                             kv->seq_len, block_len, bi, B, T_max, Hq, Hkv, D, c.rms_eps, kc, vc, kv->s_max, stream));
      TRY(tr.put(qkv, (size_t)M * qkv_w * 2));
      TRY(launch_attention(qkv, kc, vc, kv->seq_len, block_len, bi, B, T_max, Hq, Hkv, D, kv->s_max, attn, att,
                           ws.att_bytes, stream));
      TRY(tr.put(attn, (size_t)M * Hq * D * 2));
      TRY(launch_f16_rows(attn, M, (int64_t)Hq * D, attn16, inv_a, stream));
      TRY(launch_umma_w8a16_prepared(attn16, inv_a, reinterpret_cast<const int8_t*>(L.o_w), L.o_delta, M, H, (int64_t)Hq * D, x,
                                     false, x, partial, false, status, stream));
      umma_w8a16_plan(M, H, (int64_t)Hq * D, &ns, &mpad);
      TRY(launch_reduce_residual_rmsnorm_f16(partial, ns, mpad, inv_a, L.o_delta, x,
                                             reinterpret_cast<const __nv_bfloat16*>(L.mlp_norm), M, H, c.rms_eps, h, h16, inv_h,
                                             stream));
      TRY(tr.put(x, (size_t)M * H * 2));
      TRY(launch_umma_w8a16_prepared(h16, inv_h, reinterpret_cast<const int8_t*>(L.gateup_w), L.gateup_delta, M, 2 * (int64_t)F, H,
                                     gu, false, nullptr, partial, true, status, stream));
      TRY(launch_swiglu_f16(gu, M, F, act, act16, inv_f, stream));
      TRY(tr.put(act, (size_t)M * F * 2));
      TRY(launch_umma_w8a16_prepared(act16, inv_f, reinterpret_cast<const int8_t*>(L.down_w), L.down_delta, M, H, F, x, false, x,
                                     partial, false, status, stream));
      umma_w8a16_plan(M, H, F, &ns, &mpad);
      TRY(launch_reduce_residual_rmsnorm_f16(partial, ns, mpad, inv_f, L.down_delta, x, norm_of(l + 1), M, H, c.rms_eps, h, h16,
                                             inv_h, stream));
      TRY(tr.put(x, (size_t)M * H * 2));
    }
    TRY(tr.put(h, (size_t)M * H * 2));
    TRY(launch_umma_w8a16_prepared(h16, inv_h, reinterpret_cast<const int8_t*>(m->w.lm_w), m->w.lm_delta, M, c.vocab, H, logits,
                                   true, nullptr, partial, true, status, stream));
    TRY(launch_argmax(logits, M, c.vocab, top1, reinterpret_cast<unsigned long long*>(wsp + ws.keys), stream));
    TRY(launch_accept(tokens, parents, block_len, top1, bi, B, T_max, accept_len, bonus, accept_path, stream));
    return QUASAR_OK;
  }

  // W8A8: the norm and SwiGLU kernels smooth and quantise their output rows themselves (Eq. 9), straight into the place
  // where the linear layer that follows keeps its quantised operand; that layer is then called without an input.
  const bool a8_fuse = a8 && M <= kMaxRowsPerGemm && H <= 8192 && F <= 24576;
  auto norm = [&](const __nv_bfloat16* in, const void* gain, const float* smooth) -> int {
    if (!a8_fuse) return launch_rmsnorm(in, reinterpret_cast<const __nv_bfloat16*>(gain), M, H, c.rms_eps, h, stream);
    int8_t* xq = nullptr;
    float* dxp = nullptr;
    linear_w8a8_operand_slots(lin, M, H, &xq, &dxp);
    return launch_rmsnorm_q8(in, reinterpret_cast<const __nv_bfloat16*>(gain), smooth, M, H, c.rms_eps, h, xq, dxp, stream);
  };
  for (int l = 0; l < c.n_layers; ++l) {
    const quasar_layer_weights& L = m->layers[l];
    __nv_bfloat16* kc = reinterpret_cast<__nv_bfloat16*>(kv->k) + (size_t)l * layer_stride;
    __nv_bfloat16* vc = reinterpret_cast<__nv_bfloat16*>(kv->v) + (size_t)l * layer_stride;
    TRY(norm(x, L.attn_norm, L.qkv_smooth));
    TRY(tr.put(h, (size_t)M * H * 2));
    TRY(linear(a8_fuse ? nullptr : h, L.qkv_w, L.qkv_delta, L.qkv_smooth, qkv_w, H, qkv, false, nullptr));
    TRY(tr.put(qkv, (size_t)M * qkv_w * 2));
    TRY(launch_rope_append(qkv, reinterpret_cast<const __nv_bfloat16*>(c.qk_norm ? L.q_norm : nullptr),
                           reinterpret_cast<const __nv_bfloat16*>(c.qk_norm ? L.k_norm : nullptr), m->rope_table,
                           kv->seq_len, block_len, bi, B, T_max, Hq, Hkv, D, c.rms_eps, kc, vc, kv->s_max, stream));
    TRY(tr.put(qkv, (size_t)M * qkv_w * 2));
    TRY(launch_attention(qkv, kc, vc, kv->seq_len, block_len, bi, B, T_max, Hq, Hkv, D, kv->s_max, attn, att,
                         ws.att_bytes, stream));
    TRY(tr.put(attn, (size_t)M * Hq * D * 2));
    TRY(linear(attn, L.o_w, L.o_delta, L.o_smooth, H, Hq * D, x, false, x));
    TRY(tr.put(x, (size_t)M * H * 2));
    TRY(norm(x, L.mlp_norm, L.gateup_smooth));
    TRY(linear(a8_fuse ? nullptr : h, L.gateup_w, L.gateup_delta, L.gateup_smooth, 2 * F, H, gu, false, nullptr));
    if (a8_fuse) {
      int8_t* xq = nullptr;
      float* dxp = nullptr;
      linear_w8a8_operand_slots(lin, M, F, &xq, &dxp);
      TRY(launch_swiglu_q8(gu, L.down_smooth, M, F, act, xq, dxp, stream));
    } else {
      TRY(launch_swiglu(gu, M, F, act, stream));
    }
    TRY(tr.put(act, (size_t)M * F * 2));
    TRY(linear(a8_fuse ? nullptr : act, L.down_w, L.down_delta, L.down_smooth, H, F, x, false, x));
    TRY(tr.put(x, (size_t)M * H * 2));
  }
  TRY(norm(x, m->w.final_norm, m->w.lm_smooth));
  TRY(tr.put(h, (size_t)M * H * 2));
  TRY(linear(a8_fuse ? nullptr : h, m->w.lm_w, m->w.lm_delta, m->w.lm_smooth, c.vocab, H, logits, true, nullptr));
  TRY(launch_argmax(logits, M, c.vocab, top1, reinterpret_cast<unsigned long long*>(wsp + ws.keys), stream));
  TRY(launch_accept(tokens, parents, block_len, top1, bi, B, T_max, accept_len, bonus, accept_path, stream));
  return QUASAR_OK;
}

int plan_replay(quasar_plan* p, cudaStream_t stream) {
  if (p->exec == nullptr) {  // the pass is one persistent kernel: nothing to replay, launch it
    return verify_impl(p->model, &p->kv, p->tokens, p->parents, p->block_len, p->B, p->T_max, p->logits_out,
                       p->accept_len, p->bonus, p->accept_path, p->workspace, p->workspace_bytes, p->status, stream);
  }
  QUASAR_CUDA_CHECK(cudaGraphLaunch(p->exec, stream));
  count_launch(p->kernels);
  return QUASAR_OK;
}

}  // namespace

extern "C" {

const char* quasar_last_error(void) { return g_err; }

int64_t quasar_kernel_launches(void) { return (int64_t)g_launches.load(); }

int quasar_quantize(const void* w_bf16, int64_t N, int64_t K, int8_t* q_out, float* delta_out, void* stream) {
  if (N < 0 || K < 0) { set_error("quantize: negative size"); return QUASAR_ERR_INVALID_ARG; }
  if (N == 0 || K == 0) return QUASAR_OK;
  if (K % 8 != 0 || N > 0x7fffffffLL) { set_error("quantize: K=%lld must be a multiple of 8", (long long)K); return QUASAR_ERR_SHAPE; }
  REQUIRE_PTR(w_bf16, "w_bf16");
  REQUIRE_PTR(q_out, "q_out");
  REQUIRE_PTR(delta_out, "delta_out");
  return launch_quantize(reinterpret_cast<const __nv_bfloat16*>(w_bf16), N, K, q_out, delta_out, (cudaStream_t)stream);
}

int quasar_linear_workspace_bytes(int64_t M, int64_t N, int64_t K, size_t* bytes_out) {
  if (bytes_out == nullptr || M <= 0 || N <= 0 || K <= 0) { set_error("linear_workspace_bytes: bad argument"); return QUASAR_ERR_INVALID_ARG; }
  *bytes_out = linear_workspace_bytes(M, N, K);
  return QUASAR_OK;
}

int quasar_linear(const void* x, const void* w, const float* delta, int32_t weight_dtype, int64_t M, int64_t N,
                  int64_t K, void* y, int32_t y_is_f32, const void* residual, void* workspace, size_t workspace_bytes,
                  void* stream) {
  if (weight_dtype != QUASAR_W_INT8 && weight_dtype != QUASAR_W_BF16) { set_error("linear: weight_dtype %d", weight_dtype); return QUASAR_ERR_INVALID_ARG; }
  REQUIRE_PTR(x, "x");
  REQUIRE_PTR(w, "w");
  REQUIRE_PTR(y, "y");
  REQUIRE_PTR(workspace, "workspace");
  if (weight_dtype == QUASAR_W_INT8) REQUIRE_PTR(delta, "delta");
  if (residual && !aligned16(residual)) { set_error("residual is not 16-byte aligned"); return QUASAR_ERR_ALIGN; }
  return launch_linear(reinterpret_cast<const __nv_bfloat16*>(x), w, delta, weight_dtype, M, N, K, y, y_is_f32 != 0,
                       reinterpret_cast<const __nv_bfloat16*>(residual), workspace, workspace_bytes,
                       (cudaStream_t)stream);
}

int quasar_smoothing_factors(const float* act_absmax, const void* w_bf16, int64_t N, int64_t K, float alpha,
                             float* s_out, void* stream) {
  if (N <= 0 || K <= 0 || !(alpha >= 0.f && alpha <= 1.f)) { set_error("smoothing_factors: bad size or alpha"); return QUASAR_ERR_INVALID_ARG; }
  REQUIRE_PTR(act_absmax, "act_absmax");
  REQUIRE_PTR(w_bf16, "w_bf16");
  REQUIRE_PTR(s_out, "s_out");
  return launch_smoothing_factors(act_absmax, reinterpret_cast<const __nv_bfloat16*>(w_bf16), N, K, alpha, s_out,
                                  (cudaStream_t)stream);
}

static int quantize_smoothed_checked(const char* what, const void* v, const float* s, int mode, int64_t rows, int64_t K,
                                     int8_t* q_out, float* delta_out, void* stream) {
  if (rows < 0 || K < 0) { set_error("%s: negative size", what); return QUASAR_ERR_INVALID_ARG; }
  if (rows == 0 || K == 0) return QUASAR_OK;
  if (K % 8 != 0 || rows > 0x7fffffffLL) { set_error("%s: K=%lld must be a multiple of 8", what, (long long)K); return QUASAR_ERR_SHAPE; }
  REQUIRE_PTR(v, "input");
  REQUIRE_PTR(q_out, "q_out");
  REQUIRE_PTR(delta_out, "delta_out");
  if (s && !aligned16(s)) { set_error("%s: s is not 16-byte aligned", what); return QUASAR_ERR_ALIGN; }
  return launch_quantize_smoothed(reinterpret_cast<const __nv_bfloat16*>(v), s, mode, rows, K, q_out, delta_out,
                                  (cudaStream_t)stream);
}

int quasar_quantize_weights_smoothed(const void* w_bf16, const float* s, int64_t N, int64_t K, int8_t* q_out,
                                     float* delta_out, void* stream) {
  return quantize_smoothed_checked("quantize_weights_smoothed", w_bf16, s, 1, N, K, q_out, delta_out, stream);
}

int quasar_quantize_activations(const void* x_bf16, const float* s, int64_t M, int64_t K, int8_t* q_out,
                                float* delta_out, void* stream) {
  return quantize_smoothed_checked("quantize_activations", x_bf16, s, 2, M, K, q_out, delta_out, stream);
}

int quasar_linear_w8a8_workspace_bytes(int64_t M, int64_t N, int64_t K, size_t* bytes_out) {
  if (bytes_out == nullptr || M <= 0 || N <= 0 || K <= 0) { set_error("linear_w8a8_workspace_bytes: bad argument"); return QUASAR_ERR_INVALID_ARG; }
  *bytes_out = linear_w8a8_workspace_bytes(M, N, K);
  return QUASAR_OK;
}

int quasar_linear_w8a8(const void* x, const float* s, const int8_t* w, const float* delta_w, int64_t M, int64_t N,
                       int64_t K, void* y, int32_t y_is_f32, const void* residual, int32_t* acc_out, void* workspace,
                       size_t workspace_bytes, void* stream) {
  REQUIRE_PTR(x, "x");
  REQUIRE_PTR(w, "w");
  REQUIRE_PTR(delta_w, "delta_w");
  REQUIRE_PTR(y, "y");
  REQUIRE_PTR(workspace, "workspace");
  if (s && !aligned16(s)) { set_error("s is not 16-byte aligned"); return QUASAR_ERR_ALIGN; }
  if (residual && !aligned16(residual)) { set_error("residual is not 16-byte aligned"); return QUASAR_ERR_ALIGN; }
  if (acc_out && !aligned16(acc_out)) { set_error("acc_out is not 16-byte aligned"); return QUASAR_ERR_ALIGN; }
  return launch_linear_w8a8(reinterpret_cast<const __nv_bfloat16*>(x), s, w, delta_w, M, N, K, y, y_is_f32 != 0,
                            reinterpret_cast<const __nv_bfloat16*>(residual), acc_out, workspace, workspace_bytes, nullptr,
                            (cudaStream_t)stream);
}

int quasar_quantize_int4(const void* w_bf16, int64_t N, int64_t K, uint8_t* packed_out, float* delta_out, void* stream) {
  if (N < 0 || K < 0) { set_error("quantize_int4: negative size"); return QUASAR_ERR_INVALID_ARG; }
  if (N == 0 || K == 0) return QUASAR_OK;
  if (K % 128 != 0 || N > 0x7fffffffLL) { set_error("quantize_int4: K=%lld must be a multiple of 128", (long long)K); return QUASAR_ERR_SHAPE; }
  REQUIRE_PTR(w_bf16, "w_bf16");
  REQUIRE_PTR(packed_out, "packed_out");
  REQUIRE_PTR(delta_out, "delta_out");
  return launch_quantize_int4(reinterpret_cast<const __nv_bfloat16*>(w_bf16), N, K, packed_out, delta_out, (cudaStream_t)stream);
}

int quasar_linear_w4_workspace_bytes(int64_t M, int64_t N, int64_t K, size_t* bytes_out) {
  if (bytes_out == nullptr || M <= 0 || N <= 0 || K <= 0 || K % 128 != 0) { set_error("linear_w4_workspace_bytes: bad argument"); return QUASAR_ERR_INVALID_ARG; }
  *bytes_out = linear_w4_workspace_bytes(M, N, K);
  return QUASAR_OK;
}

int quasar_linear_w4(const void* x, const uint8_t* packed, const float* delta, int64_t M, int64_t N, int64_t K, void* y,
                     int32_t y_is_f32, const void* residual, void* workspace, size_t workspace_bytes, void* stream) {
  REQUIRE_PTR(x, "x");
  REQUIRE_PTR(packed, "packed");
  REQUIRE_PTR(delta, "delta");
  REQUIRE_PTR(y, "y");
  REQUIRE_PTR(workspace, "workspace");
  if (residual && !aligned16(residual)) { set_error("residual is not 16-byte aligned"); return QUASAR_ERR_ALIGN; }
  return launch_linear_w4(reinterpret_cast<const __nv_bfloat16*>(x), packed, delta, M, N, K, y, y_is_f32 != 0,
                          reinterpret_cast<const __nv_bfloat16*>(residual), workspace, workspace_bytes, (cudaStream_t)stream);
}

int quasar_linear_static(const void* x, const void* w, const float* delta, int32_t weight_dtype, int64_t M, int64_t N,
                         int64_t K, void* y, int32_t y_is_f32, const void* residual, void* stream) {
  if (weight_dtype != QUASAR_W_INT8 && weight_dtype != QUASAR_W_BF16) { set_error("linear_static: weight_dtype %d", weight_dtype); return QUASAR_ERR_INVALID_ARG; }
  REQUIRE_PTR(x, "x");
  REQUIRE_PTR(w, "w");
  REQUIRE_PTR(y, "y");
  if (weight_dtype == QUASAR_W_INT8) REQUIRE_PTR(delta, "delta");
  if (residual && !aligned16(residual)) { set_error("residual is not 16-byte aligned"); return QUASAR_ERR_ALIGN; }
  return launch_linear_static(reinterpret_cast<const __nv_bfloat16*>(x), w, delta, weight_dtype, M, N, K, y,
                              y_is_f32 != 0, reinterpret_cast<const __nv_bfloat16*>(residual), (cudaStream_t)stream);
}

size_t quasar_linear_static_scratch_bytes(void) { return linear_static_scratch_bytes(); }

int quasar_model_create(const quasar_config* cfg, const quasar_weights* w, quasar_model** out) {
  if (cfg == nullptr || w == nullptr || out == nullptr) { set_error("model_create: NULL argument"); return QUASAR_ERR_INVALID_ARG; }
  *out = nullptr;
  TRY(check_cfg(*cfg));
  if (cfg->n_layers > 0 && w->layers == nullptr) { set_error("model_create: layers is NULL"); return QUASAR_ERR_INVALID_ARG; }
  const bool q = cfg->weight_dtype == QUASAR_W_INT8;
  REQUIRE_PTR(w->embed, "embed");
  REQUIRE_PTR(w->final_norm, "final_norm");
  REQUIRE_PTR(w->lm_w, "lm_w");
  if (q) REQUIRE_PTR(w->lm_delta, "lm_delta");
  for (int l = 0; l < cfg->n_layers; ++l) {
    const quasar_layer_weights& L = w->layers[l];
    REQUIRE_PTR(L.attn_norm, "attn_norm");
    REQUIRE_PTR(L.qkv_w, "qkv_w");
    REQUIRE_PTR(L.o_w, "o_w");
    REQUIRE_PTR(L.mlp_norm, "mlp_norm");
    REQUIRE_PTR(L.gateup_w, "gateup_w");
    REQUIRE_PTR(L.down_w, "down_w");
    if (q) {
      REQUIRE_PTR(L.qkv_delta, "qkv_delta");
      REQUIRE_PTR(L.o_delta, "o_delta");
      REQUIRE_PTR(L.gateup_delta, "gateup_delta");
      REQUIRE_PTR(L.down_delta, "down_delta");
    }
    if (cfg->qk_norm) {
      REQUIRE_PTR(L.q_norm, "q_norm");
      REQUIRE_PTR(L.k_norm, "k_norm");
    }
  }
  quasar_model* m = new (std::nothrow) quasar_model();
  if (m == nullptr) { set_error("model_create: out of host memory"); return QUASAR_ERR_INVALID_ARG; }
  m->cfg = *cfg;
  m->w = *w;
  m->layers.assign(w->layers, w->layers + cfg->n_layers);
  m->w.layers = m->layers.data();
  const size_t tbytes = (size_t)cfg->max_seq * (cfg->head_dim / 2) * sizeof(float2);
  cudaError_t e = cudaMalloc(&m->rope_table, tbytes);
  if (e != cudaSuccess) {
    set_error("model_create: cudaMalloc(%zu) failed: %s", tbytes, cudaGetErrorString(e));
    delete m;
    return QUASAR_ERR_CUDA;
  }
  int rc = launch_rope_table(m->rope_table, cfg->max_seq, cfg->head_dim, cfg->rope_theta, 0);
  if (rc == QUASAR_OK && cudaStreamSynchronize(0) != cudaSuccess) { set_error("model_create: rope table kernel failed"); rc = QUASAR_ERR_CUDA; }
  if (rc != QUASAR_OK) {
    cudaFree(m->rope_table);
    delete m;
    return rc;
  }
  // The persistent kernel: its grid, a permuted copy of every matrix in the order each CTA streams it,
  // and the table of the GEMMs of the pass in execution order.
  int ncta = 0;
  if (cfg->act_dtype == QUASAR_A_BF16 && mega_grid_size(cfg->weight_dtype, cfg->head_dim, &ncta) == QUASAR_OK && ncta > 0 &&
      ncta <= kMaxGrid) {
    std::vector<MegaJob> jobs;
    std::vector<MegaLayer> mls;
    std::vector<const void*> src;
    const int qkv_w = (cfg->n_q_heads + 2 * cfg->n_kv_heads) * cfg->head_dim;
    for (int l = 0; l < cfg->n_layers; ++l) {
      const quasar_layer_weights& L = m->layers[l];
      jobs.push_back({nullptr, q ? L.qkv_delta : nullptr, reinterpret_cast<const __nv_bfloat16*>(L.attn_norm), qkv_w,
                      cfg->hidden, kJobQkv, 1.f});
      src.push_back(L.qkv_w);
      jobs.push_back({nullptr, q ? L.o_delta : nullptr, nullptr, cfg->hidden, cfg->n_q_heads * cfg->head_dim, kJobO, 1.f});
      src.push_back(L.o_w);
      jobs.push_back({nullptr, q ? L.gateup_delta : nullptr, reinterpret_cast<const __nv_bfloat16*>(L.mlp_norm),
                      2 * cfg->ffn, cfg->hidden, kJobGateUp, 1.f});
      src.push_back(L.gateup_w);
      jobs.push_back({nullptr, q ? L.down_delta : nullptr, nullptr, cfg->hidden, cfg->ffn, kJobDown, 1.f});
      src.push_back(L.down_w);
      mls.push_back({reinterpret_cast<const __nv_bfloat16*>(cfg->qk_norm ? L.q_norm : nullptr),
                     reinterpret_cast<const __nv_bfloat16*>(cfg->qk_norm ? L.k_norm : nullptr)});
    }
    jobs.push_back({nullptr, q ? w->lm_delta : nullptr, reinterpret_cast<const __nv_bfloat16*>(w->final_norm),
                    cfg->vocab, cfg->hidden, kJobLm, 1.f});
    src.push_back(w->lm_w);
    if (mls.empty()) mls.push_back({nullptr, nullptr});
    // Normed GEMMs feed h = x * r * gain with |x r| <= sqrt(K): a static power-of-two scale keeps h
    // inside the fp16 range whatever the activations are (1 unless a gain is in the hundreds).
    {
      std::vector<uint16_t> gh;
      for (auto& j : jobs) {
        if (j.gain == nullptr) continue;
        gh.resize(j.K);
        if (cudaMemcpy(gh.data(), j.gain, (size_t)j.K * 2, cudaMemcpyDeviceToHost) != cudaSuccess) {
          set_error("model_create: reading a norm gain failed: %s", cudaGetErrorString(cudaGetLastError()));
          quasar_model_destroy(m);
          return QUASAR_ERR_CUDA;
        }
        float gmax = 0.f;
        for (int k = 0; k < j.K; ++k) {
          const uint32_t bits = (uint32_t)gh[k] << 16;
          float f;
          memcpy(&f, &bits, 4);
          f = f < 0 ? -f : f;
          if (f > gmax) gmax = f;
        }
        const float bound = gmax * sqrtf((float)j.K) * 1.01f;
        if (bound > 32768.f && bound < 3.0e38f) {
          int e;
          (void)frexpf(bound, &e);
          j.xscale = ldexpf(1.f, 15 - e);
        }
      }
    }
    const size_t esz = q ? 1 : 2;
    size_t total = 0;
    std::vector<size_t> offs;
    for (auto& j : jobs) {
      offs.push_back(total);
      total += align_up((size_t)j.N * j.K * esz);
    }
    // weights_in_place: the caller hands the weight buffers over to the persistent kernel - every matrix is
    // permuted where it lies (through one scratch buffer of the largest matrix, freed again), no second copy is
    // kept, and the kernel-per-step form, which reads the row-major layout, is switched off for this model.
    const bool in_place = cfg->weights_in_place != 0;
    cudaError_t e2 = cudaSuccess;
    unsigned char* scratch = nullptr;
    if (in_place) {
      size_t largest = 0;
      for (auto& j : jobs) largest = std::max(largest, align_up((size_t)j.N * j.K * esz));
      e2 = cudaMalloc(&scratch, largest);
    } else {
      e2 = cudaMalloc(&m->mega_weights, total);
    }
    if (e2 == cudaSuccess) e2 = cudaMalloc(&m->mega_jobs, jobs.size() * sizeof(MegaJob));
    if (e2 == cudaSuccess) e2 = cudaMalloc(&m->mega_layers, mls.size() * sizeof(MegaLayer));
    int rc2 = QUASAR_OK;
    if (e2 == cudaSuccess) {
      for (size_t i = 0; i < jobs.size() && rc2 == QUASAR_OK; ++i) {
        if (in_place) {
          void* w = const_cast<void*>(src[i]);
          jobs[i].wp = w;
          rc2 = launch_repack(src[i], scratch, jobs[i].N, jobs[i].K, jobs[i].kind, cfg->weight_dtype, ncta, 0);
          if (rc2 == QUASAR_OK)
            e2 = cudaMemcpyAsync(w, scratch, (size_t)jobs[i].N * jobs[i].K * esz, cudaMemcpyDeviceToDevice, 0);
          if (e2 != cudaSuccess) break;
        } else {
          jobs[i].wp = m->mega_weights + offs[i];
          rc2 = launch_repack(src[i], m->mega_weights + offs[i], jobs[i].N, jobs[i].K, jobs[i].kind, cfg->weight_dtype, ncta, 0);
        }
      }
      if (rc2 == QUASAR_OK && e2 == cudaSuccess) e2 = cudaMemcpy(m->mega_jobs, jobs.data(), jobs.size() * sizeof(MegaJob), cudaMemcpyHostToDevice);
      if (rc2 == QUASAR_OK && e2 == cudaSuccess) e2 = cudaMemcpy(m->mega_layers, mls.data(), mls.size() * sizeof(MegaLayer), cudaMemcpyHostToDevice);
      if (rc2 == QUASAR_OK && e2 == cudaSuccess) e2 = cudaStreamSynchronize(0);
    }
    if (scratch) cudaFree(scratch);
    if (in_place && e2 == cudaSuccess && rc2 == QUASAR_OK) m->path = 2;
    if (e2 != cudaSuccess || rc2 != QUASAR_OK) {
      if (e2 != cudaSuccess) set_error("model_create: tables of the persistent kernel (%zu bytes): %s", total, cudaGetErrorString(e2));
      quasar_model_destroy(m);
      return e2 != cudaSuccess ? QUASAR_ERR_CUDA : rc2;
    }
    m->mega_ncta = ncta;
  }
  *out = m;
  return QUASAR_OK;
}

int quasar_set_path(quasar_model* m, int32_t path) {
  if (m == nullptr || path < 0 || path > 2) { set_error("set_path: bad argument"); return QUASAR_ERR_INVALID_ARG; }
  if (m->cfg.weights_in_place && path != 2) {
    set_error("set_path: this model's weights were permuted in place for the persistent kernel; only path 2 exists");
    return QUASAR_ERR_INVALID_ARG;
  }
  m->path = path;
  return QUASAR_OK;
}

int quasar_uses_persistent_kernel(const quasar_model* m, int32_t B, int32_t T_max) {
  if (m == nullptr || B < 1 || T_max < 1) { set_error("uses_persistent_kernel: bad argument"); return QUASAR_ERR_INVALID_ARG; }
  return uses_persistent_kernel(m, B, T_max) ? 1 : 0;
}

int quasar_set_wait_budget(quasar_model* m, uint64_t budget_ns, int32_t test_extra_arrivals) {
  if (m == nullptr || budget_ns == 0 || test_extra_arrivals < 0 || test_extra_arrivals > 1024) {
    set_error("set_wait_budget: bad argument");
    return QUASAR_ERR_INVALID_ARG;
  }
  m->wait_budget_ns = budget_ns;
  m->barrier_extra = (unsigned)test_extra_arrivals;
  return QUASAR_OK;
}

int quasar_model_destroy(quasar_model* m) {
  if (m == nullptr) return QUASAR_OK;
  if (m->mega_weights) cudaFree(m->mega_weights);
  if (m->mega_jobs) cudaFree(m->mega_jobs);
  if (m->mega_layers) cudaFree(m->mega_layers);
  if (m->rope_table) cudaFree(m->rope_table);
  delete m;
  return QUASAR_OK;
}

int quasar_workspace_bytes(const quasar_model* m, int32_t B, int32_t T_max, size_t* bytes_out) {
  if (m == nullptr || bytes_out == nullptr || B < 1 || T_max < 1 || T_max > QUASAR_MAX_BLOCK) { set_error("workspace_bytes: bad argument"); return QUASAR_ERR_INVALID_ARG; }
  *bytes_out = layout(m->cfg, B, T_max, m->cfg.max_seq).total;
  return QUASAR_OK;
}

int quasar_trace_bytes(const quasar_model* m, int32_t B, int32_t T_max, size_t* bytes_out) {
  if (m == nullptr || bytes_out == nullptr || B < 1 || T_max < 1) { set_error("trace_bytes: bad argument"); return QUASAR_ERR_INVALID_ARG; }
  const quasar_config& c = m->cfg;
  const size_t M = (size_t)B * T_max;
  const size_t qkv_w = (size_t)(c.n_q_heads + 2 * c.n_kv_heads) * c.head_dim;
  const size_t per_layer = M * 2 * ((size_t)c.hidden * 3 + qkv_w * 2 + (size_t)c.n_q_heads * c.head_dim + c.ffn);
  *bytes_out = M * c.hidden * 2 * 2 + per_layer * c.n_layers;
  return QUASAR_OK;
}

int quasar_set_trace(quasar_model* m, void* trace_buf, size_t bytes) {
  if (m == nullptr) { set_error("set_trace: model is NULL"); return QUASAR_ERR_INVALID_ARG; }
  m->trace_buf = trace_buf;
  m->trace_bytes = trace_buf ? bytes : 0;
  return QUASAR_OK;
}

int quasar_verify(quasar_model* m, const quasar_kv* kv, const int32_t* tokens, const int32_t* parents,
                  const int32_t* block_len, int32_t B, int32_t T_max, float* logits_out, int32_t* accept_len,
                  int32_t* bonus, int32_t* accept_path, void* workspace, size_t workspace_bytes, int32_t* status,
                  void* stream) {
  return verify_impl(m, kv, tokens, parents, block_len, B, T_max, logits_out, accept_len, bonus, accept_path, workspace,
                     workspace_bytes, status, (cudaStream_t)stream);
}

int quasar_ngram_draft(const int32_t* history, const int32_t* hist_len, int32_t B, int32_t S, int32_t gamma,
                       int32_t k_min, int32_t k_max, int32_t* draft, int32_t* draft_len, void* stream) {
  if (B < 1 || S < 1 || gamma < 1 || gamma > QUASAR_MAX_BLOCK - 1 || k_min < 1 || k_max < k_min) {
    set_error("ngram_draft: B=%d S=%d gamma=%d K=(%d,%d)", B, S, gamma, k_min, k_max);
    return QUASAR_ERR_INVALID_ARG;
  }
  REQUIRE_PTR(history, "history");
  REQUIRE_PTR(hist_len, "hist_len");
  REQUIRE_PTR(draft, "draft");
  REQUIRE_PTR(draft_len, "draft_len");
  return launch_ngram_draft(history, hist_len, B, S, gamma, k_min, k_max, draft, draft_len, (cudaStream_t)stream);
}

int quasar_accept_stochastic_workspace_bytes(int32_t B, int32_t T_max, size_t* bytes_out) {
  if (bytes_out == nullptr || B < 1 || T_max < 1) { set_error("accept_stochastic_workspace_bytes: bad argument"); return QUASAR_ERR_INVALID_ARG; }
  *bytes_out = accept_stochastic_workspace_bytes(B, T_max);
  return QUASAR_OK;
}

int quasar_accept_stochastic(const float* logits, const int32_t* tokens, const int32_t* block_len, const float* q_probs,
                             int32_t B, int32_t T_max, int32_t V, float temperature, const float* r_accept,
                             const float* r_sample, int32_t* accept_len, int32_t* next_token, void* workspace,
                             size_t workspace_bytes, void* stream) {
  if (B < 1 || T_max < 1 || T_max > QUASAR_MAX_BLOCK || V < 1 || B > 65535) { set_error("accept_stochastic: B=%d T_max=%d V=%d", B, T_max, V); return QUASAR_ERR_SHAPE; }
  if (!(temperature > 0.f)) { set_error("accept_stochastic: temperature must be positive (use the greedy acceptance of quasar_verify at 0)"); return QUASAR_ERR_INVALID_ARG; }
  REQUIRE_PTR(logits, "logits");
  REQUIRE_PTR(tokens, "tokens");
  REQUIRE_PTR(block_len, "block_len");
  REQUIRE_PTR(r_accept, "r_accept");
  REQUIRE_PTR(r_sample, "r_sample");
  REQUIRE_PTR(accept_len, "accept_len");
  REQUIRE_PTR(next_token, "next_token");
  REQUIRE_PTR(workspace, "workspace");
  if (q_probs && !aligned16(q_probs)) { set_error("q_probs is not 16-byte aligned"); return QUASAR_ERR_ALIGN; }
  if (workspace_bytes < accept_stochastic_workspace_bytes(B, T_max)) { set_error("accept_stochastic: workspace too small"); return QUASAR_ERR_CAPACITY; }
  return launch_accept_stochastic(logits, tokens, block_len, q_probs, B, T_max, V, temperature, r_accept, r_sample, accept_len,
                                  next_token, workspace, (cudaStream_t)stream);
}

int quasar_kv_commit(quasar_model* m, const quasar_kv* kv, const int32_t* accept_len, const int32_t* accept_path,
                     int32_t B, int32_t T_max, void* stream) {
  if (m == nullptr || kv == nullptr) { set_error("kv_commit: NULL argument"); return QUASAR_ERR_INVALID_ARG; }
  if (B < 1 || B > kv->batch || T_max < 1 || T_max > QUASAR_MAX_BLOCK) { set_error("kv_commit: B=%d T_max=%d", B, T_max); return QUASAR_ERR_SHAPE; }
  REQUIRE_PTR(kv->k, "kv.k");
  REQUIRE_PTR(kv->v, "kv.v");
  REQUIRE_PTR(kv->seq_len, "kv.seq_len");
  REQUIRE_PTR(accept_len, "accept_len");
  const quasar_config& c = m->cfg;
  return launch_kv_commit(reinterpret_cast<__nv_bfloat16*>(kv->k), reinterpret_cast<__nv_bfloat16*>(kv->v), kv->seq_len,
                          accept_len, accept_path, c.n_layers, kv->batch, B, T_max, c.n_kv_heads, c.head_dim, kv->s_max,
                          (cudaStream_t)stream);
}

int quasar_plan_create(quasar_model* m, const quasar_kv* kv, const int32_t* tokens, const int32_t* parents,
                       const int32_t* block_len, int32_t B, int32_t T_max, float* logits_out, int32_t* accept_len,
                       int32_t* bonus, int32_t* accept_path, void* workspace, size_t workspace_bytes, int32_t* status,
                       quasar_plan** out) {
  if (out == nullptr) { set_error("plan_create: out is NULL"); return QUASAR_ERR_INVALID_ARG; }
  *out = nullptr;
  if (m != nullptr && m->trace_buf != nullptr) { set_error("plan_create: switch the trace off first"); return QUASAR_ERR_INVALID_ARG; }
  cudaStream_t s;
  QUASAR_CUDA_CHECK(cudaStreamCreateWithFlags(&s, cudaStreamNonBlocking));
  quasar_plan* p = new (std::nothrow) quasar_plan();
  if (p == nullptr) { cudaStreamDestroy(s); set_error("plan_create: out of host memory"); return QUASAR_ERR_INVALID_ARG; }
  // one eager pass first: it configures kernel attributes (not allowed while capturing) and validates arguments
  int rc = verify_impl(m, kv, tokens, parents, block_len, B, T_max, logits_out, accept_len, bonus, accept_path,
                       workspace, workspace_bytes, status, s);
  if (rc == QUASAR_OK && cudaStreamSynchronize(s) != cudaSuccess) { set_error("plan_create: eager pass failed: %s", cudaGetErrorString(cudaGetLastError())); rc = QUASAR_ERR_CUDA; }
  if (rc == QUASAR_OK && !uses_persistent_kernel(m, B, T_max)) {
    const long long before = quasar_kernel_launches();
    cudaError_t e = cudaStreamBeginCapture(s, cudaStreamCaptureModeThreadLocal);
    if (e != cudaSuccess) { set_error("plan_create: begin capture: %s", cudaGetErrorString(e)); rc = QUASAR_ERR_CUDA; }
    if (rc == QUASAR_OK) {
      rc = verify_impl(m, kv, tokens, parents, block_len, B, T_max, logits_out, accept_len, bonus, accept_path,
                       workspace, workspace_bytes, status, s);
      e = cudaStreamEndCapture(s, &p->graph);
      if (rc == QUASAR_OK && e != cudaSuccess) { set_error("plan_create: end capture: %s", cudaGetErrorString(e)); rc = QUASAR_ERR_CUDA; }
    }
    p->kernels = (int)(quasar_kernel_launches() - before);
    count_launch(-p->kernels);  // captured launches did not run
    if (rc == QUASAR_OK) {
      e = cudaGraphInstantiate(&p->exec, p->graph, 0);
      if (e != cudaSuccess) { set_error("plan_create: instantiate: %s", cudaGetErrorString(e)); rc = QUASAR_ERR_CUDA; }
    }
  }
  cudaStreamDestroy(s);
  if (rc != QUASAR_OK) {
    if (p->exec) cudaGraphExecDestroy(p->exec);
    if (p->graph) cudaGraphDestroy(p->graph);
    delete p;
    return rc;
  }
  p->tokens = tokens; p->parents = parents; p->block_len = block_len;
  p->accept_len = accept_len; p->bonus = bonus; p->accept_path = accept_path; p->status = status;
  p->B = B; p->T_max = T_max;
  p->model = m; p->kv = *kv; p->logits_out = logits_out; p->workspace = workspace; p->workspace_bytes = workspace_bytes;
  *out = p;
  return QUASAR_OK;
}

int quasar_plan_launch(quasar_plan* p, void* stream) {
  if (p == nullptr) { set_error("plan_launch: plan is NULL"); return QUASAR_ERR_INVALID_ARG; }
  return plan_replay(p, (cudaStream_t)stream);
}

int quasar_plan_destroy(quasar_plan* p) {
  if (p == nullptr) return QUASAR_OK;
  if (p->exec) cudaGraphExecDestroy(p->exec);
  if (p->graph) cudaGraphDestroy(p->graph);
  delete p;
  return QUASAR_OK;
}

int quasar_plan_run_host(quasar_plan* p, const int32_t* tokens_host, const int32_t* parents_host,
                         const int32_t* block_len_host, int32_t* accept_len_host, int32_t* bonus_host,
                         int32_t* accept_path_host, int32_t* status_host, void* stream) {
  if (p == nullptr || tokens_host == nullptr) { set_error("plan_run_host: NULL argument"); return QUASAR_ERR_INVALID_ARG; }
  cudaStream_t s = (cudaStream_t)stream;
  const size_t bt = (size_t)p->B * p->T_max * sizeof(int32_t), bb = (size_t)p->B * sizeof(int32_t);
  QUASAR_CUDA_CHECK(cudaMemcpyAsync(const_cast<int32_t*>(p->tokens), tokens_host, bt, cudaMemcpyHostToDevice, s));
  if (parents_host && p->parents)
    QUASAR_CUDA_CHECK(cudaMemcpyAsync(const_cast<int32_t*>(p->parents), parents_host, bt, cudaMemcpyHostToDevice, s));
  if (block_len_host)
    QUASAR_CUDA_CHECK(cudaMemcpyAsync(const_cast<int32_t*>(p->block_len), block_len_host, bb, cudaMemcpyHostToDevice, s));
  TRY(plan_replay(p, s));
  if (accept_len_host) QUASAR_CUDA_CHECK(cudaMemcpyAsync(accept_len_host, p->accept_len, bb, cudaMemcpyDeviceToHost, s));
  if (bonus_host) QUASAR_CUDA_CHECK(cudaMemcpyAsync(bonus_host, p->bonus, bb, cudaMemcpyDeviceToHost, s));
  if (accept_path_host && p->accept_path)
    QUASAR_CUDA_CHECK(cudaMemcpyAsync(accept_path_host, p->accept_path, bt, cudaMemcpyDeviceToHost, s));
  if (status_host) QUASAR_CUDA_CHECK(cudaMemcpyAsync(status_host, p->status, sizeof(int32_t), cudaMemcpyDeviceToHost, s));
  QUASAR_CUDA_CHECK(cudaStreamSynchronize(s));
  return QUASAR_OK;
}

}  // extern "C"
