// Shared declarations of the CUDA path (never included by the CPU oracle).
#pragma once

#include <cuda_bf16.h>
#include <cuda_runtime.h>
#include <stdint.h>

#include "../../include/quasar.h"

namespace quasar {

void set_error(const char* fmt, ...);
void count_launch(int n = 1);

#define QUASAR_CUDA_CHECK(expr)                                                        \
  do {                                                                                 \
    cudaError_t e__ = (expr);                                                          \
    if (e__ != cudaSuccess) {                                                          \
      quasar::set_error("%s failed: %s (%s:%d)", #expr, cudaGetErrorString(e__), __FILE__, __LINE__); \
      return QUASAR_ERR_CUDA;                                                          \
    }                                                                                  \
  } while (0)

#define QUASAR_LAUNCH_CHECK()                                                          \
  do {                                                                                 \
    quasar::count_launch();                                                            \
    cudaError_t e__ = cudaGetLastError();                                              \
    if (e__ != cudaSuccess) {                                                          \
      quasar::set_error("kernel launch failed: %s (%s:%d)", cudaGetErrorString(e__), __FILE__, __LINE__); \
      return QUASAR_ERR_CUDA;                                                          \
    }                                                                                  \
  } while (0)

static inline bool aligned16(const void* p) { return (reinterpret_cast<uintptr_t>(p) & 15u) == 0; }

#ifdef __CUDACC__
// The fp16 form of an activation row for the tcgen05 weight-only GEMM: the row times the power of two that puts
// its largest magnitude in [2^14, 2^15), and the inverse of that power (exact both ways).
__device__ __forceinline__ void f16_row_scale(float amax, float& scale, float& inv) {
  scale = 1.f;
  inv = 1.f;
  if (amax > 0.f && amax < 3.0e38f) {
    int e;
    (void)frexpf(amax, &e);            // amax = f * 2^e, f in [0.5, 1)
    scale = ldexpf(1.f, 15 - e);
    inv = ldexpf(1.f, e - 15);
  }
}
#endif

constexpr int kMaxRowsPerGemm = 72;  // rows one skinny-GEMM launch handles (9 MMA column tiles)

// ---- launchers (each only enqueues work on `stream`) -------------------------------------------

int launch_quantize(const __nv_bfloat16* w, int64_t N, int64_t K, int8_t* q, float* delta, cudaStream_t stream);

size_t linear_workspace_bytes(int64_t M, int64_t N, int64_t K);
int launch_linear(const __nv_bfloat16* x, const void* w, const float* delta, int weight_dtype, int64_t M, int64_t N,
                  int64_t K, void* y, bool y_is_f32, const __nv_bfloat16* residual, void* workspace,
                  size_t workspace_bytes, cudaStream_t stream, int32_t* status = nullptr);

// The same launch with the split-K scratch taken from a fixed array inside the library.
size_t linear_static_scratch_bytes();
int launch_linear_static(const __nv_bfloat16* x, const void* w, const float* delta, int weight_dtype, int64_t M,
                         int64_t N, int64_t K, void* y, bool y_is_f32, const __nv_bfloat16* residual,
                         cudaStream_t stream);

// ---- W8A8 (Section 3.2 Eq. 4-8, Section 3.3 Eq. 9-10) ----
int launch_smoothing_factors(const float* act_absmax, const __nv_bfloat16* w, int64_t N, int64_t K, float alpha,
                             float* s_out, cudaStream_t stream);
// mode 1: v / s (offline weights), mode 2: v * s (activations); s == nullptr: plain
int launch_quantize_smoothed(const __nv_bfloat16* v, const float* s, int mode, int64_t rows, int64_t K, int8_t* q,
                             float* delta, cudaStream_t stream);
size_t linear_w8a8_workspace_bytes(int64_t M, int64_t N, int64_t K);
void linear_w8a8_operand_slots(void* workspace, int64_t M, int64_t K, int8_t** xq, float** dx);
int launch_linear_w8a8(const __nv_bfloat16* x, const float* smooth, const int8_t* w, const float* delta_w, int64_t M,
                       int64_t N, int64_t K, void* y, bool y_is_f32, const __nv_bfloat16* residual, int32_t* acc_out,
                       void* workspace, size_t workspace_bytes, int32_t* status, cudaStream_t stream);

// tcgen05 form of the W8A8 linear layer for blocks of 9..80 rows (umma_gemm.cu)
bool umma_w8a8_usable(int64_t M, int64_t N, int64_t K);
size_t umma_w8a8_partial_bytes(int64_t M, int64_t N, int64_t K);
int launch_umma_w8a8(const int8_t* xq, const float* dx, const int8_t* w, const float* dw, int64_t M, int64_t N, int64_t K,
                     void* y, bool y_is_f32, const __nv_bfloat16* residual, int32_t* acc_out, int* counters, void* partial,
                     int32_t* error_word, cudaStream_t stream);

bool umma_w8a16_usable(int64_t M, int64_t N, int64_t K);
size_t umma_w8a16_scratch_bytes(int64_t M, int64_t N, int64_t K);
int launch_umma_w8a16(const __nv_bfloat16* x, const int8_t* w, const float* dw, int64_t M, int64_t N, int64_t K, void* y,
                      bool y_is_f32, const __nv_bfloat16* residual, void* scratch, int32_t* error_word, cudaStream_t stream);
// the same in pieces, for a pass that lets the producer of the activations write their fp16 form and the consumer of
// the result add up the k-ranges (api.cu)
void umma_w8a16_plan(int64_t M, int64_t N, int64_t K, int* nsplit, int* mpad);
size_t umma_w8a16_partial_bytes(int64_t M, int64_t N, int64_t K);
int launch_f16_rows(const __nv_bfloat16* x, int64_t M, int64_t K, void* x16, float* inv_scale, cudaStream_t stream);
int launch_umma_w8a16_prepared(const void* x16, const float* inv, const int8_t* w, const float* dw, int64_t M, int64_t N,
                               int64_t K, void* y, bool y_is_f32, const __nv_bfloat16* residual, void* partial, bool finalize,
                               int32_t* error_word, cudaStream_t stream);

// the weight-only linear layer for at most 8 rows as an exact integer contraction on tcgen05 (umma_gemm.cu)
bool umma_rows8_usable(int64_t M, int64_t N, int64_t K);
size_t umma_rows8_scratch_bytes(int64_t M, int64_t N, int64_t K);
int launch_umma_rows8(const __nv_bfloat16* x, const int8_t* w, const float* dw, int64_t M, int64_t N, int64_t K, void* y,
                      bool y_is_f32, const __nv_bfloat16* residual, void* scratch, int32_t* error_word, cudaStream_t stream);

// stochastic acceptance of a chain (Section 3.1 Eq. 2-3)
size_t accept_stochastic_workspace_bytes(int B, int T_max);
int launch_accept_stochastic(const float* logits, const int32_t* tokens, const int32_t* block_len, const float* q_probs, int B,
                             int T_max, int V, float temperature, const float* r_accept, const float* r_sample,
                             int32_t* accept_len, int32_t* next_token, void* workspace, cudaStream_t stream);

// prompt-lookup drafter (Section 4.1)
int launch_ngram_draft(const int32_t* history, const int32_t* hist_len, int B, int S, int gamma, int k_min, int k_max,
                       int32_t* draft, int32_t* draft_len, cudaStream_t stream);

// 4-bit group-wise weights (Section 6 outlook)
int launch_quantize_int4(const __nv_bfloat16* w, int64_t N, int64_t K, uint8_t* packed, float* delta, cudaStream_t stream);
size_t linear_w4_workspace_bytes(int64_t M, int64_t N, int64_t K);
int launch_linear_w4(const __nv_bfloat16* x, const uint8_t* w, const float* delta, int64_t M, int64_t N, int64_t K, void* y,
                     bool y_is_f32, const __nv_bfloat16* residual, void* workspace, size_t workspace_bytes,
                     cudaStream_t stream);

// Per-call description of the draft blocks, derived on the device from tokens / parents / block_len.
struct BlockInfo {
  uint64_t* anc;    // [B*T_max] bit j set: block row j is row i itself or an ancestor of it
  int32_t* depth;   // [B*T_max]
  int32_t* valid;   // [B] 1 if the sequence is processed (block fits, parents well formed)
};

int launch_block_prep(const int32_t* tokens, const int32_t* parents, const int32_t* block_len, const int32_t* seq_len,
                      int B, int T_max, int s_max, int vocab, BlockInfo bi, int32_t* status, cudaStream_t stream);

int launch_embed(const int32_t* tokens, const __nv_bfloat16* embed, int M, int H, int vocab, __nv_bfloat16* x,
                 cudaStream_t stream);

int launch_rmsnorm(const __nv_bfloat16* x, const __nv_bfloat16* g, int M, int H, float eps, __nv_bfloat16* y,
                   cudaStream_t stream);

// QK-RMSNorm + RoPE on the q and k heads of qkv (in place) and K/V append at slot seq_len[b] + row.
int launch_rope_append(__nv_bfloat16* qkv, const __nv_bfloat16* q_norm, const __nv_bfloat16* k_norm,
                       const float2* rope_table, const int32_t* seq_len, const int32_t* block_len, BlockInfo bi, int B,
                       int T_max, int Hq, int Hkv, int D, float eps, __nv_bfloat16* k_cache_layer,
                       __nv_bfloat16* v_cache_layer, int s_max, cudaStream_t stream);

size_t attention_workspace_bytes(int B, int T_max, int Hq, int Hkv, int D, int s_max);
int launch_attention(const __nv_bfloat16* qkv, const __nv_bfloat16* k_cache_layer, const __nv_bfloat16* v_cache_layer,
                     const int32_t* seq_len, const int32_t* block_len, BlockInfo bi, int B, int T_max, int Hq, int Hkv,
                     int D, int s_max, __nv_bfloat16* out, void* workspace, size_t workspace_bytes,
                     cudaStream_t stream);

int launch_swiglu(const __nv_bfloat16* gu, int M, int F, __nv_bfloat16* act, cudaStream_t stream);

// Fused forms for the pass whose linear layers take a prepared fp16 operand (umma_gemm.cu): each also writes the
// fp16 form of its output rows (x16 [M][width] + inv [M]).
int launch_rmsnorm_f16(const __nv_bfloat16* x, const __nv_bfloat16* g, int M, int H, float eps, __nv_bfloat16* y, void* y16,
                       float* inv, cudaStream_t stream);
// The same for the W8A8 pass: the producer smooths and quantises its output rows per token (Eq. 9) into xq / dx.
int launch_rmsnorm_q8(const __nv_bfloat16* x, const __nv_bfloat16* g, const float* smooth, int M, int H, float eps,
                      __nv_bfloat16* y, int8_t* xq, float* dx, cudaStream_t stream);
int launch_swiglu_q8(const __nv_bfloat16* gu, const float* smooth, int M, int F, __nv_bfloat16* act, int8_t* xq, float* dx,
                     cudaStream_t stream);
int launch_swiglu_f16(const __nv_bfloat16* gu, int M, int F, __nv_bfloat16* act, void* act16, float* inv, cudaStream_t stream);
// x += bf16(dw * dx * sum of the k-range partial sums) (the epilogue of a residual linear layer), then y = RMSNorm(x) * g
// with its fp16 form: one kernel in place of the split-K reduction, the norm and the operand pre-pass
int launch_reduce_residual_rmsnorm_f16(const float* partial, int nsplit, int mpad, const float* dx, const float* dw,
                                       __nv_bfloat16* x, const __nv_bfloat16* g, int M, int H, float eps, __nv_bfloat16* y,
                                       void* y16, float* inv, cudaStream_t stream);

// keys: M x 8 bytes of scratch
int launch_argmax(const float* logits, int M, int V, int32_t* top1, unsigned long long* keys, cudaStream_t stream);

int launch_accept(const int32_t* tokens, const int32_t* parents, const int32_t* block_len, const int32_t* top1,
                  BlockInfo bi, int B, int T_max, int32_t* accept_len, int32_t* bonus, int32_t* accept_path,
                  cudaStream_t stream);

int launch_kv_commit(__nv_bfloat16* k_cache, __nv_bfloat16* v_cache, int32_t* seq_len, const int32_t* accept_len,
                     const int32_t* accept_path, int L, int B_cache, int B, int T_max, int Hkv, int D, int s_max,
                     cudaStream_t stream);

int launch_rope_table(float2* table, int max_pos, int D, float theta, cudaStream_t stream);

}  // namespace quasar
