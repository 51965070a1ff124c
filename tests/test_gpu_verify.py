"""End-to-end parity of the verification pass against the oracle on the tiny model (needs a GPU)."""
import numpy as np
import pytest
import torch

import oracle
from oracle import quasar_oracle as qo
from paper_2603_01399_b200 import binding, synth
from tests.common import (gpu_model, logits_close, margins, master_getter, oracle_greedy_continuation, oracle_model,
                          prefill_oracle)

pytestmark = pytest.mark.gpu

S_MAX = 128


def _kv_to_gpu(shape, okv, batch):
    k = torch.from_numpy(okv.k_bits.view(np.int16).copy()).view(torch.bfloat16).cuda()
    v = torch.from_numpy(okv.v_bits.view(np.int16).copy()).view(torch.bfloat16).cuda()
    sl = torch.from_numpy(okv.seq_len.copy()).cuda()
    return binding.KVCache(shape, batch, okv.s_max, k=k, v=v, seq_len=sl)


def _copy(okv):
    return oracle.KVCache(okv.k_bits.copy(), okv.v_bits.copy(), okv.seq_len.copy())


@pytest.fixture(scope="module", params=["tiny", "tiny_qknorm"])
def world(request):
    shape = synth.SHAPES[request.param]
    om = oracle_model(shape, seed=0, int8=True)
    gm = gpu_model(shape, seed=0, int8=True, max_seq=S_MAX)
    # the GPU-quantised weights are the oracle-quantised weights, bit for bit
    for l in range(shape.n_layers):
        for nm, ol in (("qkv", om.layers[l].qkv), ("o", om.layers[l].o), ("gateup", om.layers[l].gateup),
                       ("down", om.layers[l].down)):
            assert np.array_equal(gm.tensors[f"l{l}.{nm}_w"].cpu().numpy(), ol.w)
            assert np.array_equal(gm.tensors[f"l{l}.{nm}_delta"].cpu().numpy(), ol.delta)
    okv = oracle.new_kv(om, 1, S_MAX)
    toks = synth.uniform_tokens((64,), shape.vocab, synth.sub_seed(2, "tokens"))
    prefill_oracle(om, okv, toks[:63].numpy(), chunk=8)
    return shape, om, gm, okv, int(toks[63])


def _run_gpu(shape, gm, okv, tokens, parents, block_len, trace=False, path=0):
    B, T = tokens.shape
    gm.set_path(path)
    kv = _kv_to_gpu(shape, okv, okv.seq_len.shape[0])
    buf = binding.VerifyBuffers(gm, B, T, want_logits=True, tree=parents is not None)
    buf.tokens.copy_(torch.from_numpy(tokens))
    if parents is not None:
        buf.parents.copy_(torch.from_numpy(parents))
    buf.block_len.copy_(torch.from_numpy(block_len))
    tr = None
    if trace:
        tr = torch.zeros(gm.trace_bytes(B, T), dtype=torch.uint8, device="cuda")
        gm.set_trace(tr)
    try:
        binding.quasar_verify(gm, kv, buf)
        torch.cuda.synchronize()
    finally:
        gm.set_trace(None)
        gm.set_path(0)
    return kv, buf, (binding.split_trace(gm, tr, B, T) if trace else None)


def _check_against_oracle(shape, r, buf, block_len, margin=5e-2):
    B = len(block_len)
    lg = buf.logits.cpu().numpy()
    for b in range(B):
        T = int(block_len[b])
        ok, mabs, mrel = logits_close(lg[b, :T], r.logits[b, :T])
        assert ok, f"logits differ: max abs {mabs:.3e}, max rel {mrel:.3e}"
        mg = margins(r.logits[b, :T])
        g_top1 = lg[b, :T].argmax(-1)
        safe = mg > margin
        assert np.array_equal(g_top1[safe], r.top1[b, :T][safe])
        path = [int(p) for p in r.accept_path[b] if p >= 0]
        if all(safe[p] for p in path):
            assert int(buf.accept_len[b]) == int(r.accept_len[b])
            assert int(buf.bonus[b]) == int(r.bonus[b])
            assert np.array_equal(buf.accept_path[b].cpu().numpy(), r.accept_path[b])


def _compare_trace(shape, r, tr, rows):
    Hq, D = shape.n_q_heads, shape.head_dim

    # Tolerances, in bf16 half-ulps of the magnitudes involved.  This comparison runs the whole pass on both
    # sides, so a tensor inherits every rounding that went the other way upstream: one flipped element is a
    # whole ulp (2 half-ulps) before the step's own rounding is added, and RMSNorm / QK-norm spread it over a
    # row.  Measured on this test (both tiny models, kernel-per-step path): bit-identical up to the first
    # attention output; worst 1.7 there; 3.0 - 4.4 on the tensors of the second layer and the final norm;
    # act = silu(gate) * up, a product of two inherited flips, worst 8.3.  Hence 2.5 before the first
    # attention, 6 after it, 10 for act.  The cache rows written by the second layer inherit the same
    # flips (worst 3.0 with an absolute floor at the tensor's rms, which is what a dot product's error
    # scales with).
    def cmp(name, got, want, ulps=6.0, prev=None):
        # for a residual sum x = prev + term the rounding of the term (of size |x - prev|) bounds the error,
        # not the possibly cancelled sum
        got = got.float().cpu().numpy().astype(np.float64)
        mag = np.abs(want) if prev is None else np.abs(want) + np.abs(prev) + np.abs(want - prev)
        # a dot product's error is absolute at the scale of the tensor, hence the rms floor
        tol = ulps * 2.0 ** -8 * np.maximum(mag, np.sqrt(np.mean(mag ** 2))) + 1e-6
        bad = np.abs(got - want) > tol
        assert not bad.any(), f"{name}: {bad.sum()} of {bad.size} differ, worst {np.abs(got - want).max():.3e}"

    cmp("embed", tr["embed"][0], r.trace["embed.b0"], ulps=0)
    for l in range(shape.n_layers):
        early = 2.5 if l == 0 else 6.0          # nothing upstream has flipped yet in the first layer
        cmp(f"l{l}.h1", tr[f"l{l}.h1"][0], r.trace[f"l{l}.h1.b0"], ulps=early)
        cmp(f"l{l}.qkv", tr[f"l{l}.qkv"][0], r.trace[f"l{l}.qkv.b0"], ulps=early)
        cmp(f"l{l}.q", tr[f"l{l}.qkv_rope"][0][:, : Hq * D], r.trace[f"l{l}.q.b0"].reshape(rows, Hq * D), ulps=early)
        cmp(f"l{l}.attn", tr[f"l{l}.attn"][0], r.trace[f"l{l}.attn.b0"])
        x_in = r.trace["embed.b0"] if l == 0 else r.trace[f"l{l - 1}.x_mlp.b0"]
        cmp(f"l{l}.x_attn", tr[f"l{l}.x_attn"][0], r.trace[f"l{l}.x_attn.b0"], prev=x_in)
        cmp(f"l{l}.act", tr[f"l{l}.act"][0], r.trace[f"l{l}.act.b0"], ulps=10.0)   # two flipped factors + rounding
        cmp(f"l{l}.x_mlp", tr[f"l{l}.x_mlp"][0], r.trace[f"l{l}.x_mlp.b0"], prev=r.trace[f"l{l}.x_attn.b0"])
    cmp("hf", tr["hf"][0], r.trace["hf.b0"])


def test_config1_chain_block_with_trace(world):
    """Tiny decoder, 64-token prefix, chain draft of 4 = the bf16 model's greedy continuation with
    replacement probability 0.3; every intermediate tensor is compared, then logits and acceptance."""
    shape, om, gm, okv, root = world
    ob = oracle_model(shape, seed=0, int8=False)
    g = oracle_greedy_continuation(ob, okv, root, 4)
    draft = synth.corrupt_draft(torch.tensor(g), 0.3, shape.vocab, seed=2).tolist()
    tokens = np.array([[root] + draft], np.int32)
    bl = np.array([5], np.int32)
    okv2 = _copy(okv)
    r = oracle.verify(om, okv2, tokens, None, bl, want_trace=True)
    kv, buf, tr = _run_gpu(shape, gm, okv, tokens, None, bl, trace=True)
    assert int(buf.status[0]) == 0
    _compare_trace(shape, r, tr, 5)
    # K written at slots 63..67: the first layer's rows within one rounding, the second layer's with the
    # inherited flips
    P = int(okv.seq_len[0])
    gk = kv.k[:, 0, :, P:P + 5].float().cpu().numpy()
    ok_ = qo.bf16_bits_to_f64(okv2.k_bits[:, 0, :, P:P + 5])
    assert np.all(np.abs(gk[0] - ok_[0]) <= 2 * 2.0 ** -8 * np.maximum(np.abs(ok_[0]), 1e-2))
    assert np.all(np.abs(gk - ok_) <= 6 * 2.0 ** -8 * np.maximum(np.abs(ok_), np.sqrt(np.mean(ok_ ** 2))))
    assert torch.equal(kv.seq_len.cpu(), torch.from_numpy(okv.seq_len))          # verify does not commit
    _check_against_oracle(shape, r, buf, bl)
    assert 0 <= int(buf.accept_len[0]) <= 4

def test_every_tensor_of_a_twelve_row_block(world):
    """A chain of 11 drafts (12 block rows) is beyond the persistent kernel: the pass runs as one kernel per step,
    with int8 weights in its fused form (tcgen05 linear layers fed by producers that write the fp16 operand, the
    k-ranges of the residual layers added up by the following norm kernel).  Every intermediate tensor is
    compared with the oracle, at the tolerances of the 5-row test."""
    shape, om, gm, okv, root = world
    g = oracle_greedy_continuation(om, okv, root, 11)
    draft = synth.corrupt_draft(torch.tensor(g), 0.3, shape.vocab, seed=5).tolist()
    tokens = np.array([[root] + draft], np.int32)
    bl = np.array([12], np.int32)
    r = oracle.verify(om, _copy(okv), tokens, None, bl, want_trace=True)
    kv, buf, tr = _run_gpu(shape, gm, okv, tokens, None, bl, trace=True)
    assert int(buf.status[0]) == 0
    _compare_trace(shape, r, tr, 12)
    _check_against_oracle(shape, r, buf, bl)
    assert 0 <= int(buf.accept_len[0]) <= 11


def test_own_greedy_draft_fully_accepted_and_idempotent(world):
    shape, om, gm, okv, root = world
    g = oracle_greedy_continuation(om, okv, root, 5)
    tokens = np.array([[root] + g[:4]], np.int32)
    bl = np.array([5], np.int32)
    r = oracle.verify(om, _copy(okv), tokens, None, bl)
    kv, buf, _ = _run_gpu(shape, gm, okv, tokens, None, bl)
    _check_against_oracle(shape, r, buf, bl)
    first = buf.logits.clone()
    binding.quasar_verify(gm, kv, buf)                       # again on the same cache, no commit
    torch.cuda.synchronize()
    assert torch.equal(first, buf.logits)


def test_tree_block_ragged_batch_and_commit(world):
    shape, om, gm, okv1, root = world
    # batch of 3 sequences with different prefix lengths, block lengths and tree shapes
    B, T = 3, 8
    okv = oracle.new_kv(om, B, S_MAX)
    rng = np.random.default_rng(3)
    for b, plen in enumerate([63, 17, 40]):
        one = oracle.new_kv(om, 1, S_MAX)
        prefill_oracle(om, one, rng.integers(0, shape.vocab, plen), chunk=16)
        okv.k_bits[:, b] = one.k_bits[:, 0]
        okv.v_bits[:, b] = one.v_bits[:, 0]
        okv.seq_len[b] = plen
    parents = np.array([[-1, 0, 0, 1, 1, 2, 3, 5], [-1, 0, 1, 2, 0, 0, 0, 0], [-1, 0, 0, 0, 0, 1, 2, 6]], np.int32)
    bl = np.array([8, 4, 8], np.int32)
    tokens = rng.integers(0, shape.vocab, (B, T)).astype(np.int32)
    # plant the int8 model's greedy path on one branch of sequences 0 and 2
    for b, branch in ((0, [2, 5, 7]), (2, [2, 6, 7])):
        one = oracle.KVCache(okv.k_bits[:, b:b + 1].copy(), okv.v_bits[:, b:b + 1].copy(), okv.seq_len[b:b + 1].copy())
        g = oracle_greedy_continuation(om, one, int(tokens[b, 0]), 3)
        for node, t in zip(branch, g):
            tokens[b, node] = t
    okv2 = _copy(okv)
    r = oracle.verify(om, okv2, tokens, parents, bl)
    assert r.accept_len[0] >= 3 or margins(r.logits[0, :8]).min() < 5e-2
    kv, buf, _ = _run_gpu(shape, gm, okv, tokens, parents, bl)
    assert int(buf.status[0]) == 0
    _check_against_oracle(shape, r, buf, bl)
    # commit on both sides with the ORACLE's decision, then a plain decode step must agree
    buf.accept_len.copy_(torch.from_numpy(r.accept_len))
    buf.accept_path.copy_(torch.from_numpy(r.accept_path))
    binding.quasar_kv_commit(gm, kv, buf, tree=True)
    oracle.kv_commit(okv2, r.accept_len, r.accept_path)
    torch.cuda.synchronize()
    assert np.array_equal(kv.seq_len.cpu().numpy(), okv2.seq_len)
    nxt = r.bonus.reshape(B, 1).astype(np.int32)
    one = np.ones(B, np.int32)
    r2 = oracle.verify(om, okv2, nxt, None, one)
    buf2 = binding.VerifyBuffers(gm, B, 1)
    buf2.tokens.copy_(torch.from_numpy(nxt))
    buf2.block_len.copy_(torch.from_numpy(one))
    binding.quasar_verify(gm, kv, buf2)
    torch.cuda.synchronize()
    _check_against_oracle(shape, r2, buf2, one)
    binding.quasar_kv_commit(gm, kv, buf2, tree=False)          # chain commit: +1 each (nothing drafted)
    torch.cuda.synchronize()
    assert np.array_equal(kv.seq_len.cpu().numpy(), okv2.seq_len + 1)


def test_device_side_errors_set_status_and_skip(world):
    shape, om, gm, okv, root = world
    bl = np.array([5], np.int32)
    bad_tok = np.array([[root, 1, shape.vocab, 3, 4]], np.int32)
    _, buf, _ = _run_gpu(shape, gm, okv, bad_tok, None, bl)
    assert int(buf.status[0]) == -7 and int(buf.bonus[0]) == -1
    bad_par = np.array([[-1, 0, 2, 1, 1]], np.int32)
    _, buf, _ = _run_gpu(shape, gm, okv, np.array([[root, 1, 2, 3, 4]], np.int32), bad_par, bl)
    assert int(buf.status[0]) == -8
    full = _copy(okv)
    full.seq_len[0] = S_MAX - 3                                   # block of 5 does not fit
    kv, buf, _ = _run_gpu(shape, gm, full, np.array([[root, 1, 2, 3, 4]], np.int32), None, bl)
    assert int(buf.status[0]) == -3
    assert torch.equal(kv.k.cpu(), torch.from_numpy(full.k_bits.view(np.int16)).view(torch.bfloat16))


@pytest.mark.parametrize("path", [1, 2])
def test_commit_leaves_a_skipped_sequence_alone(world, path):
    """Batch of two, the second sequence carries a token outside the vocabulary: it is skipped
    (accept_len = bonus = -1), and a commit afterwards changes neither its seq_len nor its cache,
    while the good sequence is committed as usual."""
    shape, om, gm, okv1, root = world
    okv = oracle.new_kv(om, 2, S_MAX)
    for b in range(2):
        okv.k_bits[:, b] = okv1.k_bits[:, 0]
        okv.v_bits[:, b] = okv1.v_bits[:, 0]
        okv.seq_len[b] = okv1.seq_len[0]
    tokens = np.array([[root, 1, 2, 3], [root, 1, shape.vocab + 5, 3]], np.int32)
    bl = np.array([4, 4], np.int32)
    kv, buf, _ = _run_gpu(shape, gm, okv, tokens, None, bl, path=path)
    assert int(buf.status[0]) == -7
    assert int(buf.accept_len[1]) == -1 and int(buf.bonus[1]) == -1
    assert 0 <= int(buf.accept_len[0]) <= 3 and 0 <= int(buf.bonus[0]) < shape.vocab
    k_before, v_before = kv.k[:, 1].clone(), kv.v[:, 1].clone()
    binding.quasar_kv_commit(gm, kv, buf)
    torch.cuda.synchronize()
    sl = kv.seq_len.cpu().numpy()
    assert sl[1] == okv.seq_len[1], "a skipped sequence was committed"
    assert sl[0] == okv.seq_len[0] + 1 + int(buf.accept_len[0])
    assert torch.equal(kv.k[:, 1], k_before) and torch.equal(kv.v[:, 1], v_before)
    # the good sequence of the batch is what the oracle computes for it alone
    r = oracle.verify(om, _copy(okv), tokens[:1], None, bl[:1])
    ok, mabs, _ = logits_close(buf.logits[0].cpu().numpy(), r.logits[0])
    assert ok, mabs


def test_a_wait_that_cannot_complete_runs_out_and_the_next_pass_is_intact(world):
    """The bounded waits of the persistent kernel: with a budget of 3 ms and a grid barrier that expects one
    arrival more than there are thread blocks, every block's first barrier wait runs out; the kernel returns
    by itself with status TIMEOUT (nothing traps, nothing waits for ever), and an ordinary pass right
    afterwards on the same model and buffers gives the result it gave before."""
    import time
    shape, om, gm, okv, root = world
    tokens = np.array([[root, 1, 2, 3, 4]], np.int32)
    bl = np.array([5], np.int32)
    kv, good, _ = _run_gpu(shape, gm, okv, tokens, None, bl, path=2)
    assert int(good.status[0]) == 0
    gm.set_wait_budget(3_000_000, test_extra_arrivals=1)
    try:
        t0 = time.perf_counter()
        _, bad, _ = _run_gpu(shape, gm, okv, tokens, None, bl, path=2)
        elapsed = time.perf_counter() - t0
    finally:
        gm.set_wait_budget(2_000_000_000, 0)
    assert int(bad.status[0]) == -6, int(bad.status[0])
    assert elapsed < 1.0, f"the kernel took {elapsed:.2f} s to give up"
    _, again, _ = _run_gpu(shape, gm, okv, tokens, None, bl, path=2)
    assert int(again.status[0]) == 0
    assert torch.equal(again.logits, good.logits)
    assert torch.equal(again.accept_len, good.accept_len) and torch.equal(again.bonus, good.bonus)
    with pytest.raises(binding.QuasarError):
        gm.set_wait_budget(0)


def test_host_side_errors(world):
    shape, om, gm, okv, root = world
    kv = _kv_to_gpu(shape, okv, 1)
    buf = binding.VerifyBuffers(gm, 1, 5)
    small = binding.VerifyBuffers(gm, 1, 1)
    buf.workspace = small.workspace
    with pytest.raises(binding.QuasarError) as e:
        binding.quasar_verify(gm, kv, buf)
    assert e.value.code == -3
    with pytest.raises(binding.QuasarError) as e:
        binding.VerifyBuffers(gm, 1, 65)
    assert e.value.code == -1


def test_bf16_weight_sibling_matches_its_oracle(world):
    shape, om, _, okv, root = world
    ob = oracle_model(shape, seed=0, int8=False)
    gb = gpu_model(shape, seed=0, int8=False, max_seq=S_MAX)
    tokens = np.array([[root, 5, 6, 7, 8]], np.int32)
    bl = np.array([5], np.int32)
    r = oracle.verify(ob, _copy(okv), tokens, None, bl)
    _, buf, _ = _run_gpu(shape, gb, okv, tokens, None, bl)
    _check_against_oracle(shape, r, buf, bl)


def test_plan_replay_and_host_call(world):
    shape, om, gm, okv, root = world
    g = oracle_greedy_continuation(om, okv, root, 5)
    tokens = np.array([[root] + g[:2] + [1, 2]], np.int32)
    bl = np.array([5], np.int32)
    r = oracle.verify(om, _copy(okv), tokens, None, bl)
    kv = _kv_to_gpu(shape, okv, 1)
    buf = binding.VerifyBuffers(gm, 1, 5)
    plan = binding.Plan(gm, kv, buf)
    th = torch.from_numpy(tokens).pin_memory()
    al = torch.zeros(1, dtype=torch.int32).pin_memory()
    bo = torch.zeros(1, dtype=torch.int32).pin_memory()
    before = binding.kernel_launches()
    plan.run_host(th, al, bo)
    assert binding.kernel_launches() > before
    _check_against_oracle(shape, r, buf, bl)
    assert int(al[0]) == int(buf.accept_len[0]) and int(bo[0]) == int(buf.bonus[0])
    plan.close()


@pytest.mark.parametrize("path", [1, 2])
def test_both_implementations_on_a_tree_of_eight_rows(world, path):
    """One kernel per step (path 1) and the persistent single kernel (path 2) against the oracle: tree block
    of 8 rows, ragged block length, greedy path planted on one branch."""
    shape, om, gm, okv, root = world
    g = oracle_greedy_continuation(om, okv, root, 3)
    parents = np.array([[-1, 0, 0, 1, 2, 2, 4, 5]], np.int32)
    tokens = np.array([[root, 7, g[0], 9, g[1], 11, g[2], 13]], np.int32)
    for T in (8, 6):
        bl = np.array([T], np.int32)
        okv2 = _copy(okv)
        r = oracle.verify(om, okv2, tokens, parents, bl)
        kv, buf, _ = _run_gpu(shape, gm, okv, tokens, parents, bl, path=path)
        assert int(buf.status[0]) == 0
        _check_against_oracle(shape, r, buf, bl)
        P = int(okv.seq_len[0])
        gk = kv.k[:, 0, :, P:P + T].float().cpu().numpy()
        ok_ = qo.bf16_bits_to_f64(okv2.k_bits[:, 0, :, P:P + T])
        assert np.all(np.abs(gk - ok_) <= 6 * 2.0 ** -8 * np.maximum(np.abs(ok_), np.sqrt(np.mean(ok_ ** 2))))
        gv = kv.v[:, 0, :, P:P + T].float().cpu().numpy()
        ov_ = qo.bf16_bits_to_f64(okv2.v_bits[:, 0, :, P:P + T])
        assert np.all(np.abs(gv - ov_) <= 6 * 2.0 ** -8 * np.maximum(np.abs(ov_), np.sqrt(np.mean(ov_ ** 2))))


@pytest.mark.parametrize("path", [1, 2])
def test_both_implementations_batch_of_two_and_decode_step(world, path):
    shape, om, gm, okv1, root = world
    B = 2
    okv = oracle.new_kv(om, B, S_MAX)
    rng = np.random.default_rng(11)
    for b, plen in enumerate([70, 5]):
        one = oracle.new_kv(om, 1, S_MAX)
        prefill_oracle(om, one, rng.integers(0, shape.vocab, plen), chunk=16)
        okv.k_bits[:, b] = one.k_bits[:, 0]
        okv.v_bits[:, b] = one.v_bits[:, 0]
        okv.seq_len[b] = plen
    tokens = rng.integers(0, shape.vocab, (B, 4)).astype(np.int32)
    bl = np.array([4, 2], np.int32)
    r = oracle.verify(om, _copy(okv), tokens, None, bl)
    _, buf, _ = _run_gpu(shape, gm, okv, tokens, None, bl, path=path)
    assert int(buf.status[0]) == 0
    _check_against_oracle(shape, r, buf, bl)
    one = np.ones(B, np.int32)                                     # block_len 1: a plain decode step
    r = oracle.verify(om, _copy(okv), tokens[:, :1].copy(), None, one)
    _, buf, _ = _run_gpu(shape, gm, okv, tokens[:, :1].copy(), None, one, path=path)
    _check_against_oracle(shape, r, buf, one)


def test_persistent_kernel_refuses_blocks_it_cannot_hold(world):
    shape, om, gm, okv, root = world
    kv = _kv_to_gpu(shape, okv, 1)
    buf = binding.VerifyBuffers(gm, 1, 12)
    gm.set_path(2)
    try:
        with pytest.raises(binding.QuasarError) as e:
            binding.quasar_verify(gm, kv, buf)
        assert e.value.code == -2
    finally:
        gm.set_path(0)


@pytest.mark.parametrize("path", [1, 2])
def test_activations_beyond_the_fp16_range(path):
    """Gate/up weights scaled up until SiLU(gate)*up exceeds 65504: the int8 path multiplies fp16 operands,
    so such rows must go through their power-of-two scale (and the persistent kernel must fall back from
    its ready-made fp16 copy of the activations to the bf16 tensor).  bf16 holds these values without
    trouble, and so does the oracle."""
    shape = synth.SHAPES["tiny_qknorm"]
    base = master_getter(shape, 0, "cpu")

    def get(kind, layer=0):
        w = base(kind, layer)
        return (w.float() * 400.0).to(torch.bfloat16) if kind == "gateup" else w

    om = oracle.build_model(shape, lambda kind, layer: synth.bf16_bits(get(kind, layer)), int8=True)
    gm = binding.Model.from_master(shape, get, S_MAX, int8=True)
    okv = oracle.new_kv(om, 1, S_MAX)
    toks = synth.uniform_tokens((24,), shape.vocab, synth.sub_seed(2, "tokens")).numpy()
    prefill_oracle(om, okv, toks[:19], chunk=8)
    tokens = toks[19:24].reshape(1, 5).astype(np.int32)
    bl = np.array([5], np.int32)
    r = oracle.verify(om, _copy(okv), tokens, None, bl, want_trace=True)
    assert max(np.abs(r.trace[f"l{l}.act.b0"]).max() for l in range(shape.n_layers)) > 65504.0
    kv, buf, _ = _run_gpu(shape, gm, okv, tokens, None, bl, path=path)
    assert int(buf.status[0]) == 0
    got = buf.logits.cpu().numpy()[0].astype(np.float64)
    want = r.logits[0].astype(np.float64)
    assert np.isfinite(got).all()
    # the logits are as large as the activations: tolerance relative to the row's spread
    tol = 1e-2 * np.maximum(np.abs(want), want.std(axis=-1, keepdims=True)) + 2e-2
    assert np.all(np.abs(got - want) <= tol), float(np.abs(got - want).max())
    safe = margins(r.logits[0]) > 0.05 * want.std()
    assert np.array_equal(got.argmax(-1)[safe], r.top1[0][safe])


def test_full_product_tree_of_28_nodes(world):
    """The other reading of "depth 4, branching [4, 2, 1, 1]": the full product tree (4 + 8 + 8 + 8 nodes,
    29 rows with the root), one branch following the int8 model's own greedy continuation."""
    shape, om, gm, okv, root = world
    par = synth.tree_parents_full((4, 2, 1, 1))
    T = len(par)
    assert T == 29 and max(synth.depths(par)) == 4
    tokens = synth.uniform_tokens((1, T), shape.vocab, synth.sub_seed(5, "tokens")).numpy().astype(np.int32)
    tokens[0, 0] = root
    g = oracle_greedy_continuation(om, okv, root, 4)
    node = 0
    for t in g:   # walk down the LAST child at every level
        node = [i for i, q in enumerate(par) if q == node][-1]
        tokens[0, node] = t
    parents = np.array([par], np.int32)
    bl = np.array([T], np.int32)
    r = oracle.verify(om, _copy(okv), tokens, parents, bl)
    if margins(r.logits[0, :T]).min() > 5e-2:
        assert int(r.accept_len[0]) == 4
    kv, buf, _ = _run_gpu(shape, gm, okv, tokens, parents, bl)
    assert int(buf.status[0]) == 0
    _check_against_oracle(shape, r, buf, bl)
