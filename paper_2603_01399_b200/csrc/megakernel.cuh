// Parameters of the persistent single-kernel verification pass.
#pragma once

#include "common.cuh"

namespace quasar {

constexpr int kMegaWarps = 8;

enum MegaJobKind { kJobQkv = 0, kJobO = 1, kJobGateUp = 2, kJobDown = 3, kJobLm = 4 };

// One GEMM of the pass, in execution order: per layer qkv, o, gate+up, down; then the LM head.
struct MegaJob {
  const void* wp;              // [N][K] int8 or bf16, every CTA's row range permuted into its consumption order
  const float* delta;          // [N] or nullptr
  const __nv_bfloat16* gain;   // RMSNorm gain fused into the operand load, or nullptr
  int N, K, kind;
  float xscale;                // normed GEMMs, int8 weights: power-of-two scale keeping h = x r gain inside fp16 (usually 1)
};

struct MegaLayer {
  const __nv_bfloat16* q_norm;  // [D] or nullptr
  const __nv_bfloat16* k_norm;
};

struct MegaParams {
  const MegaJob* jobs;      // device array, 4 L + 1 entries
  const MegaLayer* layers;  // device array, L entries
  int n_jobs, L;
  int B, T_max, M, H, Hq, Hkv, vocab, s_max, kv_batch;
  float rms_eps;
  const __nv_bfloat16* embed;
  const float2* rope_table;
  const int32_t *tokens, *parents, *block_len, *seq_len;
  __nv_bfloat16 *k_cache, *v_cache;
  // workspace
  __nv_bfloat16 *x, *qkv, *attn, *act;
  // int8 weights: the o projection's and the down projection's operands once more as fp16 (what the MMA
  // takes), written beside the bf16 tensors by the phases that produce them
  unsigned short *attn16, *act16;
  float* logits;            // [M][V] or nullptr
  int32_t* top1;
  BlockInfo bi;
  float *o_part, *ml_part;  // attention partials
  int attn_nchunk, attn_rpad;
  float* cand_val;          // [grid][8] per-CTA arg-max candidates
  int* cand_idx;
  float* ss_part;           // [grid][8] per-CTA sums of squares of the rows of x, left by the phase that wrote x
  unsigned* attn_count;     // [L][B*Hkv] chunks of a (sequence, kv head) whose attention partial is complete
  unsigned* amax_buf;       // [n_jobs][8] row maxima (float bits) of the un-normed GEMM operands
  unsigned* barrier;        // zeroed before every launch
  unsigned long long wait_budget_ns;   // every device-side wait gives up after this long
  unsigned barrier_extra;   // 0; tests of the failure path make the grid barrier expect this many more arrivals
  int32_t *accept_len, *bonus, *accept_path, *status;
};

bool mega_supported(int M, int T_max, int Hq, int Hkv, int D);
int mega_attn_nchunk(int s_max);
int mega_attn_rpad(int T_max, int Hq, int Hkv);
int mega_grid_size(int weight_dtype, int D, int* ncta_out);
// Writes the permuted copy of one weight matrix for a grid of `ncta` CTAs (same size as the source).
int launch_repack(const void* w, void* wp, int N, int K, int kind, int weight_dtype, int ncta, cudaStream_t stream);
int launch_verify_mega(const MegaParams& p, int weight_dtype, int D, int ncta, cudaStream_t stream);

}  // namespace quasar
