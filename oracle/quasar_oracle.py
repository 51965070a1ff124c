"""CPU oracle for the quantised verification pass of Quasar (arXiv 2603.01399).

TEST INFRASTRUCTURE ONLY.  This is a plain, slow, fp64 numpy restatement of
what the method computes.  Only the tests, the smoke check and the benchmark's
CPU-baseline leg may call it; the product path (the CUDA library) never does
and shares no code, table or constant with it.

What is stated by the paper and what is a reading of it
-------------------------------------------------------
* Symmetric uniform quantisation  W_int8 = Q(W, delta_w)  (Section 3.2,
  Eq. 6-7).  The paper does not fix granularity, range or rounding; the reading
  here is one step size per output channel, delta = absmax/127, range
  [-127, 127], fp32 IEEE division and round-half-to-even, all-zero row ->
  delta = 1.
* Quantised matmul  Y ~= delta_w * (W_int8 X)  (Section 3.2 Eq. 8, Section 3.3
  Eq. 10) with the activation kept in bf16 (the weight-only case of the
  paper's W8A8; the weight traffic argument of Section 3.4 is unchanged).
* One parallel forward pass of the target model over the cached context plus
  the drafted block (Section 3.1, "Verification").
* Acceptance at temperature 0: a draft token is kept while it equals the
  verifier's top-1 prediction (Section 3.1 Eq. 2 at T=0; Section 4.5's remark
  on the top-1 prediction), then the verifier's own token is emitted.
* The rest of the decoder layer (the paper only says "non-linear layers" stay
  in high precision, Section 3.3) is the pre-norm RMSNorm / QK-RMSNorm / RoPE /
  GQA / SwiGLU decoder of the benchmark configurations.

Every tensor that crosses a kernel boundary is rounded to bf16
(round-to-nearest-even); every accumulation is fp64.

Pins (tests/test_oracle_*.py): hand-worked quantisation rows, the
|w - q*delta| <= delta/2 bound, idempotence; brute-force triple-loop matmul and
exact-integer cases; closed forms for RMSNorm / RoPE (norm preservation,
relative-position property) / attention (single key, uniform scores, dense
brute-force mask); all 2^gamma acceptance patterns; block verify == row-by-row
decode; own-greedy draft fully accepted.  The whole forward has no external
reference implementation to compare with: "parity unpinned" against any outside
implementation; it is pinned as a composition of the pinned steps plus those
end-to-end invariants.
"""
from __future__ import annotations

import math
from dataclasses import dataclass, field
from typing import Dict, List, Optional

import numpy as np

# --------------------------------------------------------------------------
# bf16 helpers
# --------------------------------------------------------------------------


def bf16_round(x) -> np.ndarray:
    """Round fp64 values to the nearest bf16-representable value (ties to even).

    bf16 keeps 8 significant bits, so a finite x with binary exponent e is
    rounded to a multiple of 2^(e-7); below the smallest normal (2^-126) the
    spacing stays 2^-133."""
    x = np.asarray(x, dtype=np.float64)
    _, e = np.frexp(x)                  # x = m * 2^e, 0.5 <= |m| < 1
    e = np.maximum(e, -125)
    ulp_exp = (e - 8).astype(np.int32)  # spacing is 2^(e-8) in frexp's convention
    y = np.ldexp(np.rint(np.ldexp(x, -ulp_exp)), ulp_exp)
    big = np.abs(y) > 3.3895313892515355e38  # largest finite bf16
    if np.any(big):
        y = np.where(big, np.copysign(np.inf, y), y)
    return y


def bf16_bits_to_f64(bits) -> np.ndarray:
    b = np.asarray(bits, dtype=np.uint16).astype(np.uint32) << np.uint32(16)
    with np.errstate(invalid="ignore"):          # signalling-NaN patterns are legal input
        return b.view(np.float32).astype(np.float64)


def bf16_bits_to_f32(bits) -> np.ndarray:
    b = np.asarray(bits, dtype=np.uint16).astype(np.uint32) << np.uint32(16)
    return b.view(np.float32)


def f64_to_bf16_bits(x) -> np.ndarray:
    """Bit patterns of bf16_round(x)."""
    y = bf16_round(x).astype(np.float32)     # exact: bf16 values are fp32 values
    return (y.view(np.uint32) >> np.uint32(16)).astype(np.uint16)


# --------------------------------------------------------------------------
# Step S0: symmetric per-output-channel quantisation (Section 3.2, Eq. 6-7)
# --------------------------------------------------------------------------


def quantize(w_f32: np.ndarray):
    """w_f32: [N][K] fp32 holding bf16 values.  Returns (q int8 [N][K], delta fp32 [N])."""
    w = np.asarray(w_f32, dtype=np.float32)
    absmax = np.max(np.abs(w), axis=1)
    delta = (absmax / np.float32(127.0)).astype(np.float32)
    delta = np.where(absmax == 0, np.float32(1.0), delta).astype(np.float32)
    r = np.rint(w / delta[:, None])          # fp32 division, half-to-even
    q = np.clip(r, -127.0, 127.0).astype(np.int8)
    return q, delta


def dequantize(q: np.ndarray, delta: np.ndarray) -> np.ndarray:
    return q.astype(np.float64) * delta.astype(np.float64)[:, None]


# --------------------------------------------------------------------------
# Step S3: quantised linear  Y = delta_w * (W_int8 X)  (Eq. 8 / Eq. 10)
# --------------------------------------------------------------------------


def linear(x: np.ndarray, w: np.ndarray, delta: Optional[np.ndarray]) -> np.ndarray:
    """x: [M][K] fp64; w: [N][K] int8 (or fp64 for the bf16-weight sibling);
    delta: fp32 [N] or None.  Returns fp64 [M][N], not yet rounded."""
    acc = x @ w.astype(np.float64).T
    if delta is not None:
        acc = acc * delta.astype(np.float64)[None, :]
    return acc


# --------------------------------------------------------------------------
# The paper's W8A8 form of the linear layer (Section 3.2 Eq. 4-8, Section 3.3 Eq. 9-10):
# smoothing, int8 activations per token, exact integer accumulation, dequantisation.
# Readings where the paper is silent: the activation step size is one per token (row of X),
# absmax / 127 with the same fp32 division, rounding and zero-row rule as the weights; the
# smoothed operands W / s and X * s are formed in fp32; the factors are computed in fp64 and
# stored as fp32, and a channel whose activation or weight maximum is zero gets s = 1.
# The paper is at odds with itself on the direction of s: Eq. 4 and Eq. 9 MULTIPLY the activations by
# s and divide the weights, while Eq. 5 prints the factor of the method it builds on, which divides the
# activations; taken together an outlier channel would be scaled UP.  Reading: Eq. 4 and Eq. 9 stand as
# printed (two places agree), and Eq. 5 gives the factor the activations are divided by, so the s of
# Eq. 4 / Eq. 9 is its reciprocal, max|W_j|^(1-alpha) / max|X_j|^alpha.  With alpha = 1/2 both smoothed
# operands then have the channel maximum sqrt(max|X_j| max|W_j|), which is the stated purpose.
# --------------------------------------------------------------------------


def smoothing_factors(act_absmax: np.ndarray, w_f32: np.ndarray, alpha: float = 0.5) -> np.ndarray:
    """Eq. 5 under the reading above: the factor X is multiplied by in Eq. 4 / Eq. 9,
    s_j = max|W_j|^(1 - alpha) / max|X_j|^alpha for input channel j.
    act_absmax: fp32 [K] calibration maxima of the layer's input; w_f32: [N][K].  Returns fp32 [K]."""
    a = np.asarray(act_absmax, dtype=np.float32).astype(np.float64)
    wmax = np.max(np.abs(np.asarray(w_f32, dtype=np.float32)), axis=0).astype(np.float64)
    ok = (a > 0) & (wmax > 0)
    with np.errstate(divide="ignore", invalid="ignore"):
        s = np.power(wmax, 1.0 - alpha) / np.power(a, alpha)
    return np.where(ok, s, 1.0).astype(np.float32)


def smooth_weights(w_f32: np.ndarray, s: np.ndarray) -> np.ndarray:
    """W diag(s)^-1 of Eq. 4 (offline weight preparation, Section 3.3), in fp32."""
    return (np.asarray(w_f32, dtype=np.float32) / np.asarray(s, dtype=np.float32)[None, :]).astype(np.float32)


def quantize_activations(x: np.ndarray, s: Optional[np.ndarray]):
    """Eq. 9: X_int8 = Q(X * s, delta_x), one step size per token.  x: [M][K] holding bf16 values;
    s: fp32 [K] or None (no smoothing).  Returns (int8 [M][K], fp32 [M])."""
    xt = np.asarray(x, dtype=np.float32)
    if s is not None:
        xt = (xt * np.asarray(s, dtype=np.float32)[None, :]).astype(np.float32)
    return quantize(xt)


def int_matmul(xq: np.ndarray, wq: np.ndarray) -> np.ndarray:
    """Y_int32 = W_int8 x X_int8 (Eq. 8 / Eq. 10), exact; returns int64 [M][N] (checked to fit int32)."""
    acc = xq.astype(np.int64) @ wq.astype(np.int64).T
    assert np.all(np.abs(acc) < 2 ** 31)
    return acc


def linear_w8a8(x: np.ndarray, s: Optional[np.ndarray], wq: np.ndarray, delta_w: np.ndarray) -> np.ndarray:
    """Y ~= Y_int32 * (delta_w * delta_x) (Eq. 10).  x: [M][K] holding bf16 values; wq: int8 [N][K] =
    Q(W diag(s)^-1, delta_w).  Returns fp64 [M][N], not yet rounded."""
    xq, delta_x = quantize_activations(x, s)
    acc = int_matmul(xq, wq)
    return acc.astype(np.float64) * (delta_w.astype(np.float64)[None, :] * delta_x.astype(np.float64)[:, None])


# --------------------------------------------------------------------------
# Steps S2, S4, S6: RMSNorm, RoPE, SwiGLU
# --------------------------------------------------------------------------


def rmsnorm(x: np.ndarray, g: np.ndarray, eps: float) -> np.ndarray:
    ms = np.mean(x * x, axis=-1, keepdims=True)
    return x / np.sqrt(ms + eps) * g


def rope(x: np.ndarray, pos: np.ndarray, theta: float) -> np.ndarray:
    """Rotate-half RoPE.  x: [..., D]; pos broadcastable to x[..., 0]."""
    d = x.shape[-1]
    half = d // 2
    inv_freq = theta ** (-2.0 * np.arange(half, dtype=np.float64) / d)
    ang = np.asarray(pos, dtype=np.float64)[..., None] * inv_freq
    c, s = np.cos(ang), np.sin(ang)
    x1, x2 = x[..., :half], x[..., half:]
    return np.concatenate([x1 * c - x2 * s, x2 * c + x1 * s], axis=-1)


def silu(x: np.ndarray) -> np.ndarray:
    return x / (1.0 + np.exp(-x))


# --------------------------------------------------------------------------
# Draft block structure
# --------------------------------------------------------------------------


def block_depths(parents: List[int]) -> List[int]:
    d = []
    for i, p in enumerate(parents):
        d.append(0 if p < 0 else d[p] + 1)
    return d


def ancestor_mask(parents: List[int]) -> np.ndarray:
    """mask[i][j] = True if block row j is row i itself or one of its ancestors."""
    t = len(parents)
    m = np.zeros((t, t), dtype=bool)
    for i in range(t):
        j = i
        while j >= 0:
            m[i, j] = True
            j = parents[j]
    return m


# --------------------------------------------------------------------------
# Step S5: attention of the block rows over cached prefix + allowed block rows
# --------------------------------------------------------------------------


def attention(q: np.ndarray, k: np.ndarray, v: np.ndarray, p_len: int, mask: np.ndarray) -> np.ndarray:
    """q: [T][G][D] (the G query heads sharing one kv head); k, v: [p_len+T][D];
    mask: [T][T] bool.  Row i sees keys 0..p_len-1 and p_len+j where mask[i][j].
    Returns fp64 [T][G][D], not yet rounded."""
    t, g, d = q.shape
    scores = np.einsum("igd,jd->igj", q, k) / math.sqrt(d)
    allowed = np.concatenate([np.ones((t, p_len), dtype=bool), mask], axis=1)
    scores = np.where(allowed[:, None, :], scores, -np.inf)
    scores = scores - np.max(scores, axis=-1, keepdims=True)
    p = np.exp(scores)
    p = p / np.sum(p, axis=-1, keepdims=True)
    return np.einsum("igj,jd->igd", p, v)


# --------------------------------------------------------------------------
# Steps S7-S8: argmax and greedy acceptance
# --------------------------------------------------------------------------


def argmax_lowest(logits_row: np.ndarray) -> int:
    return int(np.argmax(logits_row))      # numpy returns the first maximum


def accept_greedy(tokens: List[int], parents: List[int], top1: List[int]):
    """Walk from the root: at the current node take the lowest-index child whose
    token equals the verifier's top-1 at that node; stop when there is none.
    Returns (accept_len, bonus, path) with path[0] = 0 (the root)."""
    t = len(tokens)
    cur = 0
    path = [0]
    while True:
        nxt = -1
        for c in range(cur + 1, t):
            if parents[c] == cur and tokens[c] == top1[cur]:
                nxt = c
                break
        if nxt < 0:
            break
        cur = nxt
        path.append(cur)
    return len(path) - 1, int(top1[cur]), path


# --------------------------------------------------------------------------
# Model / cache containers
# --------------------------------------------------------------------------


@dataclass
class Linear:
    w: np.ndarray                    # int8 [N][K], or uint16 bf16 bits [N][K]
    delta: Optional[np.ndarray]      # fp32 [N] for int8 weights, None for bf16 weights
    act_int8: bool = False           # W8A8: the input is quantised per token (Eq. 9)
    smooth: Optional[np.ndarray] = None   # fp32 [K] smoothing factors folded into w (Eq. 4), W8A8 only

    def weight_for_matmul(self) -> np.ndarray:
        if self.delta is None:
            return bf16_bits_to_f64(self.w)
        return self.w

    def __call__(self, x: np.ndarray) -> np.ndarray:
        if self.act_int8:
            return linear_w8a8(x, self.smooth, self.w, self.delta)
        return linear(x, self.weight_for_matmul(), self.delta)


@dataclass
class Layer:
    attn_norm: np.ndarray            # fp64 [H]
    qkv: Linear
    q_norm: Optional[np.ndarray]     # fp64 [D]
    k_norm: Optional[np.ndarray]
    o: Linear
    mlp_norm: np.ndarray
    gateup: Linear                   # rows [0,F) gate, [F,2F) up
    down: Linear


@dataclass
class Model:
    n_layers: int
    hidden: int
    n_q_heads: int
    n_kv_heads: int
    head_dim: int
    ffn: int
    vocab: int
    qk_norm: bool
    rope_theta: float
    rms_eps: float
    embed_bits: np.ndarray           # uint16 [V][H]
    layers: List[Layer]
    final_norm: np.ndarray
    lm_head: Linear


@dataclass
class KVCache:
    k_bits: np.ndarray               # uint16 [L][B][Hkv][S_max][D]
    v_bits: np.ndarray
    seq_len: np.ndarray              # int32 [B]

    @property
    def s_max(self) -> int:
        return self.k_bits.shape[3]


def new_kv(model: Model, batch: int, s_max: int) -> KVCache:
    shp = (model.n_layers, batch, model.n_kv_heads, s_max, model.head_dim)
    return KVCache(np.zeros(shp, np.uint16), np.zeros(shp, np.uint16), np.zeros(batch, np.int32))


@dataclass
class VerifyResult:
    logits: np.ndarray               # fp32 [B][T_max][V]
    top1: np.ndarray                 # int32 [B][T_max]
    accept_len: np.ndarray           # int32 [B]
    bonus: np.ndarray                # int32 [B]
    accept_path: np.ndarray          # int32 [B][T_max], -1 beyond accept_len
    trace: Dict[str, np.ndarray] = field(default_factory=dict)


# --------------------------------------------------------------------------
# The verification pass (Section 3.1 "Verification", Section 3.3)
# --------------------------------------------------------------------------


def verify(model: Model, kv: KVCache, tokens: np.ndarray, parents: Optional[np.ndarray],
           block_len: np.ndarray, *, n_layers_run: Optional[int] = None,
           want_trace: bool = False, want_logits: bool = True) -> VerifyResult:
    """tokens: int32 [B][T_max]; row 0 is the last emitted token (not cached
    yet), rows 1.. are draft tokens / tree nodes.  parents: None for a chain,
    else int32 [B][T_max] with parents[b][0] = -1 and parents[b][i] < i.
    Writes K and V of every block row into cache slot seq_len[b] + i; does not
    change seq_len."""
    m = model
    B, T_max = tokens.shape
    L = m.n_layers if n_layers_run is None else n_layers_run
    G = m.n_q_heads // m.n_kv_heads
    D = m.head_dim
    logits = np.zeros((B, T_max, m.vocab), np.float32)
    top1 = np.full((B, T_max), -1, np.int32)
    accept_len = np.zeros(B, np.int32)
    bonus = np.zeros(B, np.int32)
    accept_path = np.full((B, T_max), -1, np.int32)
    trace: Dict[str, np.ndarray] = {}

    def tr(name, b, val):
        if want_trace:
            trace[f"{name}.b{b}"] = np.array(val, copy=True)

    for b in range(B):
        T = int(block_len[b])
        P = int(kv.seq_len[b])
        assert 1 <= T <= T_max and P + T <= kv.s_max
        par = list(range(-1, T - 1)) if parents is None else [int(p) for p in parents[b, :T]]
        dep = np.array(block_depths(par))
        mask = ancestor_mask(par)
        pos = P + dep
        tok = tokens[b, :T]

        x = bf16_bits_to_f64(m.embed_bits[tok])                       # S1
        tr("embed", b, x)
        for l in range(L):
            ly = m.layers[l]
            h = bf16_round(rmsnorm(x, ly.attn_norm, m.rms_eps))       # S2
            tr(f"l{l}.h1", b, h)
            qkv = bf16_round(ly.qkv(h))                               # S3
            tr(f"l{l}.qkv", b, qkv)
            q = qkv[:, : m.n_q_heads * D].reshape(T, m.n_q_heads, D)
            k = qkv[:, m.n_q_heads * D: (m.n_q_heads + m.n_kv_heads) * D].reshape(T, m.n_kv_heads, D)
            v = qkv[:, (m.n_q_heads + m.n_kv_heads) * D:].reshape(T, m.n_kv_heads, D)
            if m.qk_norm:                                             # S4
                q = rmsnorm(q, ly.q_norm, m.rms_eps)
                k = rmsnorm(k, ly.k_norm, m.rms_eps)
            q = bf16_round(rope(q, pos[:, None], m.rope_theta))
            k = bf16_round(rope(k, pos[:, None], m.rope_theta))
            tr(f"l{l}.q", b, q)
            kv.k_bits[l, b, :, P:P + T, :] = f64_to_bf16_bits(k).transpose(1, 0, 2)
            kv.v_bits[l, b, :, P:P + T, :] = f64_to_bf16_bits(v).transpose(1, 0, 2)
            att = np.zeros((T, m.n_q_heads, D))
            for hk in range(m.n_kv_heads):                            # S5
                kc = bf16_bits_to_f64(kv.k_bits[l, b, hk, :P + T])
                vc = bf16_bits_to_f64(kv.v_bits[l, b, hk, :P + T])
                att[:, hk * G:(hk + 1) * G, :] = attention(q[:, hk * G:(hk + 1) * G, :], kc, vc, P, mask)
            att = bf16_round(att).reshape(T, m.n_q_heads * D)
            tr(f"l{l}.attn", b, att)
            x = bf16_round(x + bf16_round(ly.o(att)))                 # S3 + residual
            tr(f"l{l}.x_attn", b, x)
            h2 = bf16_round(rmsnorm(x, ly.mlp_norm, m.rms_eps))       # S2
            gu = bf16_round(ly.gateup(h2))                            # S3
            act = bf16_round(silu(gu[:, : m.ffn]) * gu[:, m.ffn:])    # S6
            tr(f"l{l}.act", b, act)
            x = bf16_round(x + bf16_round(ly.down(act)))              # S3 + residual
            tr(f"l{l}.x_mlp", b, x)
        hf = bf16_round(rmsnorm(x, m.final_norm, m.rms_eps))
        tr("hf", b, hf)
        if want_logits:
            lg = m.lm_head(hf).astype(np.float32)                     # S7
            logits[b, :T] = lg
            t1 = [argmax_lowest(lg[i]) for i in range(T)]
            top1[b, :T] = t1
            n, bo, path = accept_greedy([int(t) for t in tok], par, t1)   # S8
            accept_len[b] = n
            bonus[b] = bo
            accept_path[b, : len(path)] = path
    return VerifyResult(logits, top1, accept_len, bonus, accept_path, trace)


# --------------------------------------------------------------------------
# Step S9: commit the accepted tokens to the cache
# --------------------------------------------------------------------------


def kv_commit(kv: KVCache, accept_len: np.ndarray, accept_path: Optional[np.ndarray]) -> None:
    """Chain (accept_path None): seq_len[b] += 1 + accept_len[b].  Tree: the K,V of
    the accepted node at depth d move to slot seq_len[b] + d, then the same bump."""
    B = kv.seq_len.shape[0]
    for b in range(B):
        P = int(kv.seq_len[b])
        n = int(accept_len[b])
        if accept_path is not None:
            for d in range(1, n + 1):
                j = int(accept_path[b, d])
                if j != d:
                    kv.k_bits[:, b, :, P + d, :] = kv.k_bits[:, b, :, P + j, :]
                    kv.v_bits[:, b, :, P + d, :] = kv.v_bits[:, b, :, P + j, :]
        kv.seq_len[b] = P + 1 + n


# --------------------------------------------------------------------------
# Stochastic acceptance (Section 3.1 Eq. 2-3; Section 3.3 "Lossless Rejection Sampling")
# --------------------------------------------------------------------------
# Readings where the paper is silent: the target distribution is softmax(logits / T) of the row that
# predicts the drafted token; when every draft is accepted one more token is drawn from the target
# distribution of the last row (the usual completion of the scheme; the paper stops at "concludes the
# current decoding step"); a draft distribution that is not given is the point mass on the drafted token
# (a retrieval drafter such as the paper's n-gram lookup proposes one token with certainty); random
# numbers are INPUTS (r_accept per draft position, r_sample per sequence, all in [0, 1)); a token is drawn
# from unnormalised weights w by inversion: the smallest v with w_0 + ... + w_v > r_sample * sum(w).


def softmax_t(logits_row: np.ndarray, temperature: float) -> np.ndarray:
    z = np.asarray(logits_row, dtype=np.float64) / float(temperature)
    z = z - np.max(z)
    e = np.exp(z)
    return e / np.sum(e)


def sample_by_inversion(weights: np.ndarray, u: float) -> int:
    """Smallest index v with w_0 + ... + w_v > u * sum(w) (so w_v > 0); if u is so close to 1 that rounding
    leaves none, the last index with a positive weight."""
    w = np.asarray(weights, dtype=np.float64)
    c = np.cumsum(w)
    v = int(np.searchsorted(c, u * c[-1], side="right"))
    if v >= len(w):
        v = int(np.nonzero(w > 0)[0][-1])
    return v


def accept_stochastic(logits: np.ndarray, tokens: List[int], q_probs: Optional[np.ndarray], temperature: float,
                      r_accept: np.ndarray, r_sample: float):
    """Chain block.  logits: [T][V] (row i predicts the token after block row i); tokens: T block tokens
    (row 0 the last emitted token, rows 1.. the drafts); q_probs: [T][V] draft distributions (row i the
    one draft i+1 was drawn from) or None.  Returns (accept_len, next_token)."""
    t = len(tokens)
    n = 0
    for i in range(t - 1):                                   # draft i+1 against row i (Eq. 2)
        p = softmax_t(logits[i], temperature)
        tok = int(tokens[i + 1])
        q_tok = 1.0 if q_probs is None else float(q_probs[i][tok])
        ratio = 1.0 if q_tok <= 0 else min(1.0, p[tok] / q_tok)
        if q_tok <= 0 or not (float(r_accept[i]) < ratio):
            if q_probs is None:
                resid = p.copy()
                resid[tok] = 0.0                             # max(0, p - q) with q the point mass on tok
            else:
                resid = np.maximum(0.0, p - np.asarray(q_probs[i], dtype=np.float64))   # Eq. 3
            if resid.sum() <= 0:                             # p == q exactly: nothing left to correct with
                resid = p
            return n, sample_by_inversion(resid, r_sample)
        n += 1
    return n, sample_by_inversion(softmax_t(logits[t - 1], temperature), r_sample)


# --------------------------------------------------------------------------
# Drafting by prompt lookup (Section 4.1: the n-gram drafter of all experiments; lookup range
# K = (K_min, K_max), Section 4.4 / Table 3)
# --------------------------------------------------------------------------
# The paper names the method and its two parameters only.  Reading: for n = K_max down to K_min the last n
# tokens of the sequence are searched for in the tokens before them; the most recent earlier occurrence
# that is followed by at least one token wins, and the up to gamma tokens that followed it are the draft;
# the longest n that has such an occurrence is used; no occurrence for any n -> no draft.


def ngram_draft(history: List[int], gamma: int, k_min: int, k_max: int) -> List[int]:
    h = [int(t) for t in history]
    n_hist = len(h)
    for n in range(min(k_max, n_hist - 1), k_min - 1, -1):
        if n < 1:
            break
        pattern = h[n_hist - n:]
        for start in range(n_hist - n - 1, -1, -1):          # most recent first; start + n <= n_hist - 1
            if h[start:start + n] == pattern:
                return h[start + n:start + n + gamma]
    return []


# --------------------------------------------------------------------------
# 4-bit weights (Section 6, "Ultra-low Bit Verification": the first item of the paper's outlook)
# --------------------------------------------------------------------------
# The paper only names the direction (weights of 4 bits or fewer).  Reading: the operator Q of Eq. 6 with a
# range of [-7, 7] and one step size per output channel AND group of 128 consecutive input channels
# (per-channel steps alone are too coarse at 4 bits); two codes per byte, the even input channel in the low
# nibble, two's complement.


INT4_GROUP = 128


def quantize_int4(w_f32: np.ndarray, group: int = INT4_GROUP):
    """w_f32: [N][K] fp32 holding bf16 values, K a multiple of `group`.
    Returns (codes int8 [N][K] in [-7, 7], delta fp32 [N][K / group])."""
    w = np.asarray(w_f32, dtype=np.float32)
    n, k = w.shape
    assert k % group == 0
    wg = w.reshape(n, k // group, group)
    absmax = np.max(np.abs(wg), axis=2)
    delta = (absmax / np.float32(7.0)).astype(np.float32)
    delta = np.where(absmax == 0, np.float32(1.0), delta).astype(np.float32)
    q = np.clip(np.rint(wg / delta[:, :, None]), -7.0, 7.0).astype(np.int8)
    return q.reshape(n, k), delta


def pack_int4(codes: np.ndarray) -> np.ndarray:
    """int8 [N][K] in [-8, 7] -> uint8 [N][K / 2]: channel 2j in the low nibble, 2j + 1 in the high one."""
    c = codes.astype(np.int16) & 0xF
    return (c[:, 0::2] | (c[:, 1::2] << 4)).astype(np.uint8)


def unpack_int4(packed: np.ndarray) -> np.ndarray:
    p = packed.astype(np.int16)
    lo, hi = p & 0xF, (p >> 4) & 0xF
    out = np.empty((packed.shape[0], packed.shape[1] * 2), np.int16)
    out[:, 0::2], out[:, 1::2] = lo, hi
    return np.where(out >= 8, out - 16, out).astype(np.int8)


def linear_int4(x: np.ndarray, codes: np.ndarray, delta: np.ndarray, group: int = INT4_GROUP) -> np.ndarray:
    """Y[m][n] = sum_g delta[n][g] * sum_{k in g} X[m][k] * codes[n][k]  (Eq. 8 with one step per group), fp64."""
    m, k = x.shape
    n = codes.shape[0]
    xg = np.asarray(x, np.float64).reshape(m, k // group, group)
    cg = codes.astype(np.float64).reshape(n, k // group, group)
    part = np.einsum("mgk,ngk->mng", xg, cg)
    return np.einsum("mng,ng->mn", part, delta.astype(np.float64))
