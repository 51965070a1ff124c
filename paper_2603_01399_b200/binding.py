"""ctypes binding of libquasar.so: same names as the C ABI, argument marshalling only.

PyTorch is used for device memory and the current CUDA stream; every step of the
verification pass runs inside the library's kernels.  There is no CPU fallback: if
the library has not been built, `lib()` raises.
"""
from __future__ import annotations

import ctypes as C
import os
from typing import Dict, List, Optional

import torch

_HERE = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(_HERE, "libquasar.so")

QUASAR_W_INT8 = 0
QUASAR_W_BF16 = 1
QUASAR_A_BF16 = 0
QUASAR_A_INT8 = 1
QUASAR_MAX_BLOCK = 64

ERROR_NAMES = {0: "OK", -1: "INVALID_ARG", -2: "SHAPE", -3: "CAPACITY", -4: "ALIGN", -5: "CUDA", -6: "TIMEOUT",
               -7: "TOKEN", -8: "TREE"}


class QuasarError(RuntimeError):
    def __init__(self, code: int, msg: str):
        super().__init__(f"quasar error {code} ({ERROR_NAMES.get(code, '?')}): {msg}")
        self.code = code


class Config(C.Structure):
    _fields_ = [("n_layers", C.c_int32), ("hidden", C.c_int32), ("n_q_heads", C.c_int32), ("n_kv_heads", C.c_int32),
                ("head_dim", C.c_int32), ("ffn", C.c_int32), ("vocab", C.c_int32), ("qk_norm", C.c_int32),
                ("rope_theta", C.c_float), ("rms_eps", C.c_float), ("weight_dtype", C.c_int32),
                ("max_seq", C.c_int32), ("act_dtype", C.c_int32), ("weights_in_place", C.c_int32)]


class LayerWeights(C.Structure):
    _fields_ = [(n, C.c_void_p) for n in
                ("attn_norm", "qkv_w", "qkv_delta", "q_norm", "k_norm", "o_w", "o_delta", "mlp_norm", "gateup_w",
                 "gateup_delta", "down_w", "down_delta", "qkv_smooth", "o_smooth", "gateup_smooth", "down_smooth")]


class Weights(C.Structure):
    _fields_ = [("embed", C.c_void_p), ("layers", C.POINTER(LayerWeights)), ("final_norm", C.c_void_p),
                ("lm_w", C.c_void_p), ("lm_delta", C.c_void_p), ("lm_smooth", C.c_void_p)]


class KV(C.Structure):
    _fields_ = [("k", C.c_void_p), ("v", C.c_void_p), ("seq_len", C.c_void_p), ("batch", C.c_int32),
                ("s_max", C.c_int32)]


_lib = None

_vp, _i32, _i64, _sz = C.c_void_p, C.c_int32, C.c_int64, C.c_size_t
_verify_args = [_vp, C.POINTER(KV), _vp, _vp, _vp, _i32, _i32, _vp, _vp, _vp, _vp, _vp, _sz, _vp]
SIGNATURES = {
    "quasar_last_error": (C.c_char_p, []),
    "quasar_kernel_launches": (_i64, []),
    "quasar_quantize": (C.c_int, [_vp, _i64, _i64, _vp, _vp, _vp]),
    "quasar_linear_workspace_bytes": (C.c_int, [_i64, _i64, _i64, C.POINTER(_sz)]),
    "quasar_linear": (C.c_int, [_vp, _vp, _vp, _i32, _i64, _i64, _i64, _vp, _i32, _vp, _vp, _sz, _vp]),
    "quasar_smoothing_factors": (C.c_int, [_vp, _vp, _i64, _i64, C.c_float, _vp, _vp]),
    "quasar_quantize_weights_smoothed": (C.c_int, [_vp, _vp, _i64, _i64, _vp, _vp, _vp]),
    "quasar_quantize_activations": (C.c_int, [_vp, _vp, _i64, _i64, _vp, _vp, _vp]),
    "quasar_linear_w8a8_workspace_bytes": (C.c_int, [_i64, _i64, _i64, C.POINTER(_sz)]),
    "quasar_linear_w8a8": (C.c_int, [_vp, _vp, _vp, _vp, _i64, _i64, _i64, _vp, _i32, _vp, _vp, _vp, _sz, _vp]),
    "quasar_quantize_int4": (C.c_int, [_vp, _i64, _i64, _vp, _vp, _vp]),
    "quasar_linear_w4_workspace_bytes": (C.c_int, [_i64, _i64, _i64, C.POINTER(_sz)]),
    "quasar_linear_w4": (C.c_int, [_vp, _vp, _vp, _i64, _i64, _i64, _vp, _i32, _vp, _vp, _sz, _vp]),
    "quasar_linear_static_scratch_bytes": (_sz, []),
    "quasar_linear_static": (C.c_int, [_vp, _vp, _vp, _i32, _i64, _i64, _i64, _vp, _i32, _vp, _vp]),
    "quasar_model_create": (C.c_int, [C.POINTER(Config), C.POINTER(Weights), C.POINTER(_vp)]),
    "quasar_model_destroy": (C.c_int, [_vp]),
    "quasar_workspace_bytes": (C.c_int, [_vp, _i32, _i32, C.POINTER(_sz)]),
    "quasar_verify": (C.c_int, _verify_args + [_vp]),
    "quasar_ngram_draft": (C.c_int, [_vp, _vp, _i32, _i32, _i32, _i32, _i32, _vp, _vp, _vp]),
    "quasar_accept_stochastic_workspace_bytes": (C.c_int, [_i32, _i32, C.POINTER(_sz)]),
    "quasar_accept_stochastic": (C.c_int, [_vp, _vp, _vp, _vp, _i32, _i32, _i32, C.c_float, _vp, _vp, _vp, _vp, _vp, _sz, _vp]),
    "quasar_kv_commit": (C.c_int, [_vp, C.POINTER(KV), _vp, _vp, _i32, _i32, _vp]),
    "quasar_plan_create": (C.c_int, _verify_args + [C.POINTER(_vp)]),
    "quasar_plan_launch": (C.c_int, [_vp, _vp]),
    "quasar_plan_destroy": (C.c_int, [_vp]),
    "quasar_plan_run_host": (C.c_int, [_vp, _vp, _vp, _vp, _vp, _vp, _vp, _vp, _vp]),
    "quasar_trace_bytes": (C.c_int, [_vp, _i32, _i32, C.POINTER(_sz)]),
    "quasar_set_trace": (C.c_int, [_vp, _vp, _sz]),
    "quasar_set_path": (C.c_int, [_vp, _i32]),
    "quasar_set_wait_budget": (C.c_int, [_vp, C.c_uint64, _i32]),
    "quasar_uses_persistent_kernel": (C.c_int, [_vp, _i32, _i32]),
}


def lib() -> C.CDLL:
    """Loads the CUDA library; raises if it has not been built (there is no fallback)."""
    global _lib
    if _lib is None:
        if not os.path.exists(LIB_PATH):
            raise RuntimeError(f"{LIB_PATH} is missing: build it with `python -m paper_2603_01399_b200.build`")
        l = C.CDLL(LIB_PATH)
        for name, (res, args) in SIGNATURES.items():
            fn = getattr(l, name)
            fn.restype = res
            fn.argtypes = args
        _lib = l
    return _lib


def _check(rc: int) -> None:
    if rc != 0:
        raise QuasarError(rc, lib().quasar_last_error().decode())


def _ptr(t: Optional[torch.Tensor]):
    return None if t is None else t.data_ptr()


def _stream() -> int:
    return torch.cuda.current_stream().cuda_stream


def kernel_launches() -> int:
    return int(lib().quasar_kernel_launches())


# ------------------------------------------------------------------------------------------
def quasar_quantize(w_bf16: torch.Tensor):
    """bf16 [N][K] on the device -> (int8 [N][K], fp32 [N])."""
    assert w_bf16.is_cuda and w_bf16.dtype == torch.bfloat16 and w_bf16.is_contiguous() and w_bf16.dim() == 2
    n, k = w_bf16.shape
    q = torch.empty((n, k), dtype=torch.int8, device=w_bf16.device)
    d = torch.empty((n,), dtype=torch.float32, device=w_bf16.device)
    _check(lib().quasar_quantize(_ptr(w_bf16), n, k, _ptr(q), _ptr(d), _stream()))
    return q, d


def quasar_linear_workspace_bytes(m: int, n: int, k: int) -> int:
    out = _sz(0)
    _check(lib().quasar_linear_workspace_bytes(m, n, k, C.byref(out)))
    return int(out.value)


def quasar_linear(x: torch.Tensor, w: torch.Tensor, delta: Optional[torch.Tensor], residual=None, out_f32=False,
                  workspace: Optional[torch.Tensor] = None, out: Optional[torch.Tensor] = None) -> torch.Tensor:
    """x bf16 [M][K]; w int8 or bf16 [N][K]; delta fp32 [N] (int8 weights)."""
    assert x.is_cuda and x.dtype == torch.bfloat16 and x.is_contiguous() and w.is_contiguous()
    m, k = x.shape
    n = w.shape[0]
    wd = QUASAR_W_INT8 if w.dtype == torch.int8 else QUASAR_W_BF16
    if out is None:
        out = torch.empty((m, n), dtype=torch.float32 if out_f32 else torch.bfloat16, device=x.device)
    if workspace is None:
        workspace = torch.zeros(max(quasar_linear_workspace_bytes(m, n, k), 16), dtype=torch.uint8, device=x.device)
    _check(lib().quasar_linear(_ptr(x), _ptr(w), _ptr(delta), wd, m, n, k, _ptr(out), 1 if out_f32 else 0,
                               _ptr(residual), _ptr(workspace), workspace.numel(), _stream()))
    return out


def quasar_smoothing_factors(act_absmax: torch.Tensor, w_bf16: torch.Tensor, alpha: float = 0.5) -> torch.Tensor:
    """fp32 [K] calibration maxima + bf16 [N][K] weights -> fp32 [K] smoothing factors (Eq. 5)."""
    assert act_absmax.is_cuda and act_absmax.dtype == torch.float32 and w_bf16.dtype == torch.bfloat16
    n, k = w_bf16.shape
    s = torch.empty(k, dtype=torch.float32, device=w_bf16.device)
    _check(lib().quasar_smoothing_factors(_ptr(act_absmax), _ptr(w_bf16), n, k, alpha, _ptr(s), _stream()))
    return s


def quasar_quantize_weights_smoothed(w_bf16: torch.Tensor, s: Optional[torch.Tensor]):
    """Q(W diag(s)^-1, delta_w): bf16 [N][K] (+ fp32 [K]) -> (int8 [N][K], fp32 [N])."""
    n, k = w_bf16.shape
    q = torch.empty((n, k), dtype=torch.int8, device=w_bf16.device)
    d = torch.empty((n,), dtype=torch.float32, device=w_bf16.device)
    _check(lib().quasar_quantize_weights_smoothed(_ptr(w_bf16), _ptr(s), n, k, _ptr(q), _ptr(d), _stream()))
    return q, d


def quasar_quantize_activations(x_bf16: torch.Tensor, s: Optional[torch.Tensor]):
    """Q(X * s, delta_x) per token: bf16 [M][K] (+ fp32 [K]) -> (int8 [M][K], fp32 [M])."""
    m, k = x_bf16.shape
    q = torch.empty((m, k), dtype=torch.int8, device=x_bf16.device)
    d = torch.empty((m,), dtype=torch.float32, device=x_bf16.device)
    _check(lib().quasar_quantize_activations(_ptr(x_bf16), _ptr(s), m, k, _ptr(q), _ptr(d), _stream()))
    return q, d


def quasar_linear_w8a8(x: torch.Tensor, s: Optional[torch.Tensor], w: torch.Tensor, delta_w: torch.Tensor, residual=None,
                       out_f32=False, want_acc=False):
    """x bf16 [M][K]; s fp32 [K] or None; w int8 [N][K]; delta_w fp32 [N].  Returns y (and the int32
    accumulators when want_acc)."""
    m, k = x.shape
    n = w.shape[0]
    y = torch.empty((m, n), dtype=torch.float32 if out_f32 else torch.bfloat16, device=x.device)
    acc = torch.empty((m, n), dtype=torch.int32, device=x.device) if want_acc else None
    nbytes = _sz(0)
    _check(lib().quasar_linear_w8a8_workspace_bytes(m, n, k, C.byref(nbytes)))
    ws = torch.zeros(int(nbytes.value), dtype=torch.uint8, device=x.device)
    _check(lib().quasar_linear_w8a8(_ptr(x), _ptr(s), _ptr(w), _ptr(delta_w), m, n, k, _ptr(y), 1 if out_f32 else 0,
                                    _ptr(residual), _ptr(acc), _ptr(ws), ws.numel(), _stream()))
    return (y, acc) if want_acc else y


def quasar_quantize_int4(w_bf16: torch.Tensor):
    """bf16 [N][K] (K a multiple of 128) -> (packed uint8 [N][K/2], delta fp32 [N][K/128])."""
    n, k = w_bf16.shape
    packed = torch.empty((n, k // 2), dtype=torch.uint8, device=w_bf16.device)
    delta = torch.empty((n, k // 128), dtype=torch.float32, device=w_bf16.device)
    _check(lib().quasar_quantize_int4(_ptr(w_bf16), n, k, _ptr(packed), _ptr(delta), _stream()))
    return packed, delta


def quasar_linear_w4(x: torch.Tensor, packed: torch.Tensor, delta: torch.Tensor, residual=None, out_f32=False,
                     workspace=None, out=None) -> torch.Tensor:
    m, k = x.shape
    n = packed.shape[0]
    if out is None:
        out = torch.empty((m, n), dtype=torch.float32 if out_f32 else torch.bfloat16, device=x.device)
    if workspace is None:
        nbytes = _sz(0)
        _check(lib().quasar_linear_w4_workspace_bytes(m, n, k, C.byref(nbytes)))
        workspace = torch.empty(max(int(nbytes.value), 16), dtype=torch.uint8, device=x.device)
    _check(lib().quasar_linear_w4(_ptr(x), _ptr(packed), _ptr(delta), m, n, k, _ptr(out), 1 if out.dtype == torch.float32 else 0,
                                  _ptr(residual), _ptr(workspace), workspace.numel(), _stream()))
    return out


def quasar_linear_static_scratch_bytes() -> int:
    return int(lib().quasar_linear_static_scratch_bytes())


def quasar_linear_static(x: torch.Tensor, w: torch.Tensor, delta: Optional[torch.Tensor], out: torch.Tensor,
                         residual=None) -> torch.Tensor:
    """quasar_linear without a workspace argument: the library's built-in scratch array is used and
    nothing is allocated by the call (the caller supplies `out`: bf16 or fp32 [M][N])."""
    assert x.is_cuda and x.dtype == torch.bfloat16 and x.is_contiguous() and w.is_contiguous() and out.is_contiguous()
    m, k = x.shape
    n = w.shape[0]
    assert tuple(out.shape) == (m, n) and out.dtype in (torch.float32, torch.bfloat16)
    wd = QUASAR_W_INT8 if w.dtype == torch.int8 else QUASAR_W_BF16
    _check(lib().quasar_linear_static(_ptr(x), _ptr(w), _ptr(delta), wd, m, n, k, _ptr(out),
                                      1 if out.dtype == torch.float32 else 0, _ptr(residual), _stream()))
    return out


# ------------------------------------------------------------------------------------------
class Model:
    """Owns the device weight tensors (keeps them alive) and the library's model handle.

    `tensors` maps names to device tensors: embed, final_norm, lm_w, lm_delta and per layer l
    `l{l}.attn_norm`, `.qkv_w`, `.qkv_delta`, `.q_norm`, `.k_norm`, `.o_w`, `.o_delta`, `.mlp_norm`,
    `.gateup_w`, `.gateup_delta`, `.down_w`, `.down_delta` (deltas absent for bf16 weights)."""

    def __init__(self, shape, tensors: Dict[str, torch.Tensor], max_seq: int, weight_dtype: int = QUASAR_W_INT8,
                 act_dtype: int = QUASAR_A_BF16, weights_in_place: bool = False):
        self.shape = shape
        self.tensors = tensors
        self.weight_dtype = weight_dtype
        self.act_dtype = act_dtype
        self.max_seq = max_seq
        self.cfg = Config(shape.n_layers, shape.hidden, shape.n_q_heads, shape.n_kv_heads, shape.head_dim, shape.ffn,
                          shape.vocab, 1 if shape.qk_norm else 0, shape.rope_theta, shape.rms_eps, weight_dtype,
                          max_seq, act_dtype, 1 if weights_in_place else 0)
        layers = (LayerWeights * max(shape.n_layers, 1))()
        for l in range(shape.n_layers):
            for name, _ in LayerWeights._fields_:
                setattr(layers[l], name, _ptr(tensors.get(f"l{l}.{name}")))
        self._layers = layers
        w = Weights(_ptr(tensors["embed"]), layers, _ptr(tensors["final_norm"]), _ptr(tensors["lm_w"]),
                    _ptr(tensors.get("lm_delta")), _ptr(tensors.get("lm_smooth")))
        handle = _vp()
        _check(lib().quasar_model_create(C.byref(self.cfg), C.byref(w), C.byref(handle)))
        self.handle = handle
        self._trace = None

    @classmethod
    def from_master(cls, shape, get_master, max_seq: int, int8: bool = True, device="cuda", act_int8: bool = False,
                    get_act_absmax=None, alpha: float = 0.5, weights_in_place: bool = False):
        """get_master(kind, layer) -> bf16 master tensor (any device).  int8=True quantises every
        matrix on the GPU with quasar_quantize (the offline weight preparation).  act_int8=True builds the
        W8A8 verifier: get_act_absmax(kind, layer) -> fp32 [K] calibration maxima of the layer's input give
        the smoothing factors (quasar_smoothing_factors), which are folded into the weights before they are
        quantised (quasar_quantize_weights_smoothed) and kept for the online activation smoothing."""
        t: Dict[str, torch.Tensor] = {}
        assert int8 or not act_int8

        def put_linear(prefix, kind, layer):
            w = get_master(kind, layer).to(device)
            if int8 and act_int8:
                s = None
                if get_act_absmax is not None:
                    s = quasar_smoothing_factors(get_act_absmax(kind, layer).to(device), w, alpha)
                    t[prefix + "_smooth"] = s
                t[prefix + "_w"], t[prefix + "_delta"] = quasar_quantize_weights_smoothed(w, s)
            elif int8:
                q, d = quasar_quantize(w)
                t[prefix + "_w"], t[prefix + "_delta"] = q, d
            else:
                t[prefix + "_w"] = w

        t["embed"] = get_master("embed", 0).to(device)
        t["final_norm"] = get_master("final_norm", 0).to(device)
        put_linear("lm", "lm_head", 0)
        for l in range(shape.n_layers):
            t[f"l{l}.attn_norm"] = get_master("attn_norm", l).to(device)
            t[f"l{l}.mlp_norm"] = get_master("mlp_norm", l).to(device)
            if shape.qk_norm:
                t[f"l{l}.q_norm"] = get_master("q_norm", l).to(device)
                t[f"l{l}.k_norm"] = get_master("k_norm", l).to(device)
            put_linear(f"l{l}.qkv", "qkv", l)
            put_linear(f"l{l}.o", "o", l)
            put_linear(f"l{l}.gateup", "gateup", l)
            put_linear(f"l{l}.down", "down", l)
        torch.cuda.synchronize()
        return cls(shape, t, max_seq, QUASAR_W_INT8 if int8 else QUASAR_W_BF16,
                   QUASAR_A_INT8 if act_int8 else QUASAR_A_BF16, weights_in_place)

    def workspace_bytes(self, batch: int, t_max: int) -> int:
        out = _sz(0)
        _check(lib().quasar_workspace_bytes(self.handle, batch, t_max, C.byref(out)))
        return int(out.value)

    def trace_bytes(self, batch: int, t_max: int) -> int:
        out = _sz(0)
        _check(lib().quasar_trace_bytes(self.handle, batch, t_max, C.byref(out)))
        return int(out.value)

    def set_trace(self, buf: Optional[torch.Tensor]) -> None:
        self._trace = buf
        _check(lib().quasar_set_trace(self.handle, _ptr(buf), 0 if buf is None else buf.numel() * buf.element_size()))

    def set_path(self, path: int) -> None:
        """0 automatic, 1 one kernel per step, 2 persistent single-kernel pass."""
        _check(lib().quasar_set_path(self.handle, path))

    def launch_kind(self, batch: int, t_max: int) -> str:
        """How quasar_verify runs a block of this size (for reports)."""
        persistent = int(lib().quasar_uses_persistent_kernel(self.handle, batch, t_max)) == 1
        return "one persistent cooperative kernel per step" if persistent else "one kernel per step, replayed as a CUDA graph"

    def set_wait_budget(self, budget_ns: int, test_extra_arrivals: int = 0) -> None:
        """Bound of every device-side wait of the persistent kernel (default 2 s)."""
        _check(lib().quasar_set_wait_budget(self.handle, budget_ns, test_extra_arrivals))

    def weight_bytes(self) -> int:
        return sum(v.numel() * v.element_size() for k, v in self.tensors.items()
                   if k.endswith("_w") or k.endswith("_delta"))

    def close(self) -> None:
        if self.handle is not None:
            lib().quasar_model_destroy(self.handle)
            self.handle = None

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass


class KVCache:
    """bf16 K and V [L][B][Hkv][S_max][D] and int32 seq_len [B] on the device."""

    def __init__(self, shape, batch: int, s_max: int, device="cuda", k=None, v=None, seq_len=None):
        dims = (shape.n_layers, batch, shape.n_kv_heads, s_max, shape.head_dim)
        self.k = torch.zeros(dims, dtype=torch.bfloat16, device=device) if k is None else k
        self.v = torch.zeros(dims, dtype=torch.bfloat16, device=device) if v is None else v
        assert tuple(self.k.shape) == dims and tuple(self.v.shape) == dims
        self.seq_len = torch.zeros(batch, dtype=torch.int32, device=device) if seq_len is None else seq_len
        self.batch, self.s_max = batch, s_max
        self.c = KV(_ptr(self.k), _ptr(self.v), _ptr(self.seq_len), batch, s_max)


class VerifyBuffers:
    """Device buffers of one verify call (inputs, outputs, workspace)."""

    def __init__(self, model: Model, batch: int, t_max: int, want_logits: bool = True, tree: bool = False,
                 device="cuda"):
        self.batch, self.t_max = batch, t_max
        self.tokens = torch.zeros((batch, t_max), dtype=torch.int32, device=device)
        self.parents = torch.zeros((batch, t_max), dtype=torch.int32, device=device) if tree else None
        self.block_len = torch.full((batch,), t_max, dtype=torch.int32, device=device)
        self.logits = torch.zeros((batch, t_max, model.shape.vocab), dtype=torch.float32, device=device) \
            if want_logits else None
        self.accept_len = torch.zeros(batch, dtype=torch.int32, device=device)
        self.bonus = torch.zeros(batch, dtype=torch.int32, device=device)
        self.accept_path = torch.zeros((batch, t_max), dtype=torch.int32, device=device)
        self.status = torch.zeros(4, dtype=torch.int32, device=device)
        self.workspace = torch.zeros(model.workspace_bytes(batch, t_max), dtype=torch.uint8, device=device)

    def args(self, model: Model, kv: KVCache):
        return (model.handle, C.byref(kv.c), _ptr(self.tokens), _ptr(self.parents), _ptr(self.block_len), self.batch,
                self.t_max, _ptr(self.logits), _ptr(self.accept_len), _ptr(self.bonus), _ptr(self.accept_path),
                _ptr(self.workspace), self.workspace.numel(), _ptr(self.status))


def quasar_verify(model: Model, kv: KVCache, buf: VerifyBuffers) -> None:
    """Enqueues one verification pass on the current stream; results land in `buf`."""
    _check(lib().quasar_verify(*buf.args(model, kv), _stream()))


def quasar_kv_commit(model: Model, kv: KVCache, buf: VerifyBuffers, tree: bool = False) -> None:
    _check(lib().quasar_kv_commit(model.handle, C.byref(kv.c), _ptr(buf.accept_len),
                                  _ptr(buf.accept_path) if tree else None, buf.batch, buf.t_max, _stream()))


def quasar_ngram_draft(history: torch.Tensor, hist_len: torch.Tensor, gamma: int, k_min: int, k_max: int):
    """history int32 [B][S], hist_len int32 [B] -> (draft int32 [B][gamma], draft_len int32 [B])."""
    b, s = history.shape
    draft = torch.empty((b, gamma), dtype=torch.int32, device=history.device)
    dlen = torch.empty(b, dtype=torch.int32, device=history.device)
    _check(lib().quasar_ngram_draft(_ptr(history), _ptr(hist_len), b, s, gamma, k_min, k_max, _ptr(draft), _ptr(dlen), _stream()))
    return draft, dlen


def quasar_accept_stochastic(logits: torch.Tensor, tokens: torch.Tensor, block_len: torch.Tensor, q_probs, temperature: float,
                             r_accept: torch.Tensor, r_sample: torch.Tensor):
    """logits fp32 [B][T][V]; tokens int32 [B][T]; block_len int32 [B]; q_probs fp32 [B][T][V] or None;
    r_accept fp32 [B][T]; r_sample fp32 [B].  Returns (accept_len, next_token), int32 [B]."""
    b, t, v = logits.shape
    accept_len = torch.empty(b, dtype=torch.int32, device=logits.device)
    nxt = torch.empty(b, dtype=torch.int32, device=logits.device)
    nbytes = _sz(0)
    _check(lib().quasar_accept_stochastic_workspace_bytes(b, t, C.byref(nbytes)))
    ws = torch.empty(int(nbytes.value), dtype=torch.uint8, device=logits.device)
    _check(lib().quasar_accept_stochastic(_ptr(logits), _ptr(tokens), _ptr(block_len), _ptr(q_probs), b, t, v, temperature,
                                          _ptr(r_accept), _ptr(r_sample), _ptr(accept_len), _ptr(nxt), _ptr(ws), ws.numel(),
                                          _stream()))
    return accept_len, nxt


class Plan:
    """A verify pass captured into a CUDA graph by the library."""

    def __init__(self, model: Model, kv: KVCache, buf: VerifyBuffers):
        self.model, self.kv, self.buf = model, kv, buf
        h = _vp()
        _check(lib().quasar_plan_create(*buf.args(model, kv), C.byref(h)))
        self.handle = h

    def launch(self) -> None:
        _check(lib().quasar_plan_launch(self.handle, _stream()))

    def run_host(self, tokens_host: torch.Tensor, accept_len_host: torch.Tensor, bonus_host: torch.Tensor,
                 block_len_host=None, parents_host=None, accept_path_host=None, status_host=None) -> None:
        """Host (pinned) buffers in, host buffers out; returns after the stream has drained."""
        _check(lib().quasar_plan_run_host(self.handle, _ptr(tokens_host), _ptr(parents_host), _ptr(block_len_host),
                                          _ptr(accept_len_host), _ptr(bonus_host), _ptr(accept_path_host),
                                          _ptr(status_host), _stream()))

    def close(self) -> None:
        if self.handle is not None:
            lib().quasar_plan_destroy(self.handle)
            self.handle = None

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass


def split_trace(model: Model, buf_bytes: torch.Tensor, batch: int, t_max: int) -> Dict[str, torch.Tensor]:
    """Cuts a trace buffer into named bf16 tensors [B][T_max][width] in the order the library writes them."""
    s = model.shape
    m = batch * t_max
    qkv_w = s.qkv_dim
    flat = buf_bytes.view(torch.bfloat16)
    out: Dict[str, torch.Tensor] = {}
    off = 0

    def take(name, width):
        nonlocal off
        out[name] = flat[off: off + m * width].view(batch, t_max, width)
        off += m * width

    take("embed", s.hidden)
    for l in range(s.n_layers):
        take(f"l{l}.h1", s.hidden)
        take(f"l{l}.qkv", qkv_w)
        take(f"l{l}.qkv_rope", qkv_w)
        take(f"l{l}.attn", s.q_dim)
        take(f"l{l}.x_attn", s.hidden)
        take(f"l{l}.act", s.ffn)
        take(f"l{l}.x_mlp", s.hidden)
    take("hf", s.hidden)
    return out
