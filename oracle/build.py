"""Assemble an oracle Model from bf16 master tensors given as uint16 bit arrays.

TEST INFRASTRUCTURE ONLY.  `get_bits(kind, layer)` is supplied by the caller
(it usually closes over the seeded input generator); this file knows nothing
about how the numbers were drawn."""
from __future__ import annotations

from typing import Callable

import numpy as np

from . import quasar_oracle as qo


def _linear(bits: np.ndarray, int8: bool) -> qo.Linear:
    if int8:
        q, delta = qo.quantize(qo.bf16_bits_to_f32(bits))   # Section 3.3 "Offline Weight Preparation"
        return qo.Linear(q, delta)
    return qo.Linear(np.ascontiguousarray(bits), None)


def build_model(shape, get_bits: Callable[[str, int], np.ndarray], int8: bool = True) -> qo.Model:
    """shape: any object with n_layers, hidden, n_q_heads, n_kv_heads, head_dim,
    ffn, vocab, qk_norm, rope_theta, rms_eps attributes."""
    layers = []
    for l in range(shape.n_layers):
        layers.append(qo.Layer(
            attn_norm=qo.bf16_bits_to_f64(get_bits("attn_norm", l)),
            qkv=_linear(get_bits("qkv", l), int8),
            q_norm=qo.bf16_bits_to_f64(get_bits("q_norm", l)) if shape.qk_norm else None,
            k_norm=qo.bf16_bits_to_f64(get_bits("k_norm", l)) if shape.qk_norm else None,
            o=_linear(get_bits("o", l), int8),
            mlp_norm=qo.bf16_bits_to_f64(get_bits("mlp_norm", l)),
            gateup=_linear(get_bits("gateup", l), int8),
            down=_linear(get_bits("down", l), int8),
        ))
    return qo.Model(
        n_layers=shape.n_layers, hidden=shape.hidden, n_q_heads=shape.n_q_heads,
        n_kv_heads=shape.n_kv_heads, head_dim=shape.head_dim, ffn=shape.ffn, vocab=shape.vocab,
        qk_norm=bool(shape.qk_norm), rope_theta=float(shape.rope_theta), rms_eps=float(shape.rms_eps),
        embed_bits=np.ascontiguousarray(get_bits("embed", 0)),
        layers=layers,
        final_norm=qo.bf16_bits_to_f64(get_bits("final_norm", 0)),
        lm_head=_linear(get_bits("lm_head", 0), int8),
    )
