"""Stochastic acceptance on the GPU against the oracle (Section 3.1 Eq. 2-3), through the C ABI."""
import numpy as np
import pytest
import torch

from oracle import quasar_oracle as qo
from paper_2603_01399_b200 import binding

pytestmark = pytest.mark.gpu


def _oracle_margins(logits, tokens, q, temp, r_accept, r_sample):
    """The oracle's decision plus how far each of its comparisons is from its threshold (relative)."""
    n, tok = qo.accept_stochastic(logits, list(tokens), q, temp, r_accept, r_sample)
    margin = 1.0
    t = len(tokens)
    for i in range(min(n + 1, t - 1)):
        p = qo.softmax_t(logits[i], temp)
        qt = 1.0 if q is None else float(q[i][tokens[i + 1]])
        ratio = min(1.0, p[tokens[i + 1]] / qt) if qt > 0 else 0.0
        margin = min(margin, abs(float(r_accept[i]) - ratio))
    if n < t - 1:
        p = qo.softmax_t(logits[n], temp)
        w = p.copy()
        if q is None:
            w[tokens[n + 1]] = 0.0
        else:
            w = np.maximum(0.0, p - q[n])
    else:
        w = qo.softmax_t(logits[t - 1], temp)
    c = np.cumsum(w)
    tgt = r_sample * c[-1]
    edges = np.concatenate([[0.0], c])
    margin_draw = float(np.min(np.abs(edges - tgt)) / c[-1])
    return n, tok, margin, margin_draw, w


@pytest.mark.parametrize("V,with_q,temp", [(16, True, 1.0), (1000, True, 0.7), (1024, False, 1.0), (151936, False, 1.0),
                                           (32000, True, 1.3)])
def test_stochastic_acceptance_matches_the_oracle(V, with_q, temp):
    rng = np.random.default_rng(V + int(with_q))
    B, T = 24, 6
    logits = (rng.normal(size=(B, T, V)) * 2.5).astype(np.float32)
    q = None
    tokens = rng.integers(0, V, (B, T)).astype(np.int32)
    if with_q:
        # drafter: a softened copy of the target; drafts drawn from it so that acceptance is frequent
        ql = logits.astype(np.float64) * 0.8 + rng.normal(size=(B, T, V)) * 0.5
        q = np.exp(ql - ql.max(-1, keepdims=True))
        q = (q / q.sum(-1, keepdims=True)).astype(np.float32)
        for b in range(B):
            for i in range(T - 1):
                tokens[b, i + 1] = qo.sample_by_inversion(q[b, i].astype(np.float64), rng.random())
    else:
        for b in range(B):                           # point-mass drafter: often the target's top choice
            for i in range(T - 1):
                if rng.random() < 0.7:
                    tokens[b, i + 1] = int(np.argmax(logits[b, i]))
    bl = rng.integers(1, T + 1, B).astype(np.int32)
    bl[0], bl[1] = T, 1
    r_accept = rng.random((B, T)).astype(np.float32)
    r_sample = rng.random(B).astype(np.float32)
    r_sample[2] = np.float32(1.0) - np.float32(2.0 ** -24)     # as close to 1 as fp32 gets
    acc, nxt = binding.quasar_accept_stochastic(torch.from_numpy(logits).cuda(), torch.from_numpy(tokens).cuda(),
                                                torch.from_numpy(bl).cuda(), None if q is None else torch.from_numpy(q).cuda(),
                                                temp, torch.from_numpy(r_accept).cuda(), torch.from_numpy(r_sample).cuda())
    acc, nxt = acc.cpu().numpy(), nxt.cpu().numpy()
    checked = 0
    for b in range(B):
        Tb = int(bl[b])
        qb = None if q is None else q[b, :Tb].astype(np.float64)
        n, tok, m_acc, m_draw, w = _oracle_margins(logits[b, :Tb].astype(np.float64), tokens[b, :Tb], qb, temp,
                                                   r_accept[b].astype(np.float64), float(r_sample[b]))
        assert 0 <= acc[b] <= Tb - 1 and 0 <= nxt[b] < V
        if m_acc > 1e-4:                             # every accept / reject comparison is clear of its threshold
            assert acc[b] == n, (b, acc[b], n)
            assert w[nxt[b]] > 0, "a token of zero weight was drawn"
            # inversion: the drawn token's interval of the cumulative weights must hold r_sample * total, up to the
            # rounding of an fp32 running sum over V terms; where the target is clear of every edge the token is
            # the oracle's
            c = np.cumsum(w)
            tgt, tol = float(r_sample[b]) * c[-1], 3e-5 * c[-1]
            lo = c[nxt[b] - 1] if nxt[b] > 0 else 0.0
            assert lo - tol <= tgt <= c[nxt[b]] + tol, (b, nxt[b], tok, lo, tgt, c[nxt[b]])
            if m_draw > 1e-4:
                assert nxt[b] == tok, (b, nxt[b], tok)
            checked += 1
    assert checked >= B // 2


def test_stochastic_acceptance_repeats_bit_for_bit_and_accepts_everything_when_q_equals_p():
    rng = np.random.default_rng(5)
    B, T, V = 8, 5, 4096
    logits = (rng.normal(size=(B, T, V)) * 2).astype(np.float32)
    p = np.exp(logits.astype(np.float64) - logits.max(-1, keepdims=True))
    p = (p / p.sum(-1, keepdims=True))
    tokens = rng.integers(0, V, (B, T)).astype(np.int32)
    for b in range(B):
        for i in range(T - 1):
            tokens[b, i + 1] = qo.sample_by_inversion(p[b, i], rng.random())
    args = (torch.from_numpy(logits).cuda(), torch.from_numpy(tokens).cuda(), torch.full((B,), T, dtype=torch.int32, device="cuda"),
            torch.from_numpy((p * (1 + 1e-3)).astype(np.float32)).cuda(), 1.0,        # q a hair above p: ratio just below 1
            torch.from_numpy((rng.random((B, T)) * 0.99).astype(np.float32)).cuda(), torch.from_numpy(rng.random(B).astype(np.float32)).cuda())
    a1, n1 = binding.quasar_accept_stochastic(*args)
    a2, n2 = binding.quasar_accept_stochastic(*args)
    assert torch.equal(a1, a2) and torch.equal(n1, n2)
    assert (a1 == T - 1).all()
