"""Assemble an oracle Model from bf16 master tensors given as uint16 bit arrays.

TEST INFRASTRUCTURE ONLY.  `get_bits(kind, layer)` is supplied by the caller
(it usually closes over the seeded input generator); this file knows nothing
about how the numbers were drawn."""
from __future__ import annotations

from typing import Callable, Optional

import numpy as np

from . import quasar_oracle as qo


def quantize_rows_in_parallel(w_f32: np.ndarray, workers: int = 0):
    """qo.quantize applied to blocks of rows on a thread pool (every row is quantised on its own, so
    the result is the one call's; numpy releases the interpreter lock inside its loops).  For building
    full-size models in reasonable time."""
    import os
    from concurrent.futures import ThreadPoolExecutor
    workers = workers or min(32, os.cpu_count() or 1)
    n = w_f32.shape[0]
    step = max(64, -(-n // (4 * workers)))
    blocks = [(i, min(n, i + step)) for i in range(0, n, step)]
    with ThreadPoolExecutor(workers) as ex:
        parts = list(ex.map(lambda b: qo.quantize(w_f32[b[0]:b[1]]), blocks))
    return np.concatenate([p[0] for p in parts], axis=0), np.concatenate([p[1] for p in parts])


def build_model(shape, get_bits: Callable[[str, int], np.ndarray], int8: bool = True, act_int8: bool = False,
                get_act_absmax: Optional[Callable[[str, int], np.ndarray]] = None, alpha: float = 0.5,
                parallel: bool = False) -> qo.Model:
    """shape: any object with n_layers, hidden, n_q_heads, n_kv_heads, head_dim,
    ffn, vocab, qk_norm, rope_theta, rms_eps attributes.
    act_int8: the paper's W8A8 verifier (Section 3.2-3.3): every linear layer quantises its input per
    token; get_act_absmax(kind, layer) -> fp32 [K] calibration maxima of that layer's input, from which
    the smoothing factors (Eq. 5, migration strength alpha) are derived and folded into the weights before
    they are quantised (None: no smoothing)."""
    assert int8 or not act_int8

    def _linear(kind: str, layer: int) -> qo.Linear:
        bits = get_bits(kind, layer)
        if not int8:
            return qo.Linear(np.ascontiguousarray(bits), None)
        w = qo.bf16_bits_to_f32(bits)
        s = None
        if act_int8 and get_act_absmax is not None:
            s = qo.smoothing_factors(get_act_absmax(kind, layer), w, alpha)
            w = qo.smooth_weights(w, s)
        q, delta = quantize_rows_in_parallel(w) if parallel else qo.quantize(w)   # Section 3.3 "Offline Weight Preparation"
        return qo.Linear(q, delta, act_int8=act_int8, smooth=s)

    layers = []
    for l in range(shape.n_layers):
        layers.append(qo.Layer(
            attn_norm=qo.bf16_bits_to_f64(get_bits("attn_norm", l)),
            qkv=_linear("qkv", l),
            q_norm=qo.bf16_bits_to_f64(get_bits("q_norm", l)) if shape.qk_norm else None,
            k_norm=qo.bf16_bits_to_f64(get_bits("k_norm", l)) if shape.qk_norm else None,
            o=_linear("o", l),
            mlp_norm=qo.bf16_bits_to_f64(get_bits("mlp_norm", l)),
            gateup=_linear("gateup", l),
            down=_linear("down", l),
        ))
    return qo.Model(
        n_layers=shape.n_layers, hidden=shape.hidden, n_q_heads=shape.n_q_heads,
        n_kv_heads=shape.n_kv_heads, head_dim=shape.head_dim, ffn=shape.ffn, vocab=shape.vocab,
        qk_norm=bool(shape.qk_norm), rope_theta=float(shape.rope_theta), rms_eps=float(shape.rms_eps),
        embed_bits=np.ascontiguousarray(get_bits("embed", 0)),
        layers=layers,
        final_norm=qo.bf16_bits_to_f64(get_bits("final_norm", 0)),
        lm_head=_linear("lm_head", 0),
    )
