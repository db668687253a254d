"""ctypes binding of libd2c.so: argument marshalling only, same names as include/d2c.h.

torch is used for device memory and streams; every step of the path runs in the
library's kernels.  Loading fails loudly when the library has not been built.
"""
from __future__ import annotations

import ctypes as C
import os
from typing import Dict, List, Optional, Sequence

import torch

HERE = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(HERE, "libd2c.so")

N_PHASES = 13
D2C_OK, D2C_EINVAL, D2C_ESHAPE, D2C_ECAPACITY, D2C_ECUDA, D2C_ETIMEOUT = 0, -1, -2, -3, -4, -5

# every symbol include/d2c.h declares
SYMBOLS = ["d2c_workspace_bytes", "d2c_create", "d2c_step", "d2c_step_host", "d2c_commit", "d2c_state_ptrs",
           "d2c_sync_status", "d2c_last_error", "d2c_destroy", "d2c_profile", "d2c_profile_read", "d2c_phase_name", "d2c_op_select_scratch_bytes", "d2c_op_select",
           "d2c_op_gemm", "d2c_op_attention", "d2c_op_lm_head_scratch_bytes", "d2c_op_lm_head",
           "d2c_op_rollout_scratch_bytes", "d2c_op_rollout", "d2c_op_rollout_static", "d2c_op_wait_probe"]


class D2cError(RuntimeError):
    def __init__(self, code: int, msg: str):
        super().__init__(f"d2c error {code}: {msg}")
        self.code = code


class Config(C.Structure):
    _fields_ = [(n, C.c_int32) for n in ("n_layers", "d_model", "n_q_heads", "n_kv_heads", "head_dim", "d_ffn", "vocab",
                                         "max_batch", "max_seq")] + \
               [("rope_base", C.c_float), ("rms_eps", C.c_float), ("sigma", C.c_float)] + \
               [(n, C.c_int32) for n in ("qkv_bias", "stage2_candidates", "rollout_layers", "flags")]


class Weights(C.Structure):
    _fields_ = [(n, C.POINTER(C.c_void_p)) for n in ("wqkv", "bqkv", "wo", "w_gate", "w_up", "w_down", "g_attn", "g_ffn")] + \
               [("g_final", C.c_void_p), ("w_lm", C.c_void_p)]


class StepArgs(C.Structure):
    _fields_ = [("batch", C.c_int32), ("seq_len", C.c_int32), ("h0", C.c_void_p), ("mask", C.c_void_p),
                ("forced", C.c_void_p), ("forced_off", C.c_void_p), ("k", C.c_int32), ("p", C.c_float),
                ("override_key", C.c_void_p), ("override_c", C.c_void_p), ("block_lo", C.c_int32), ("block_hi", C.c_int32)]


class StepOut(C.Structure):
    _fields_ = [("sel_idx", C.c_void_p), ("row_off", C.c_void_p), ("hidden_out", C.c_void_p), ("logits", C.c_void_p),
                ("layer_in", C.c_void_p)]


class HostOut(C.Structure):
    _fields_ = [("sel_idx_host", C.c_void_p), ("row_off_host", C.c_void_p), ("hidden_out_host", C.c_void_p),
                ("conf_host", C.c_void_p), ("pred_host", C.c_void_p)]


class State(C.Structure):
    _fields_ = [(n, C.c_void_p) for n in ("kcache", "vcache", "conf", "pred", "c", "key", "sel_idx", "row_off",
                                          "lm_rows", "lm_off", "abar", "lse", "status", "gemm_clocks")]


_lib = None


def load() -> C.CDLL:
    """Loads libd2c.so; raises if it is missing (there is no fallback path)."""
    global _lib
    if _lib is not None:
        return _lib
    if not os.path.exists(LIB_PATH):
        raise RuntimeError(f"{LIB_PATH} not found: build it with `python -m paper_2509_23094_b200.build`")
    lib = C.CDLL(LIB_PATH)
    vp, i32, f32, sz = C.c_void_p, C.c_int32, C.c_float, C.c_size_t
    lib.d2c_workspace_bytes.restype = sz
    lib.d2c_workspace_bytes.argtypes = [C.POINTER(Config)]
    lib.d2c_create.argtypes = [C.POINTER(Config), C.POINTER(Weights), vp, sz, vp, C.POINTER(vp)]
    lib.d2c_step.argtypes = [vp, C.POINTER(StepArgs), C.POINTER(StepOut)]
    lib.d2c_step_host.argtypes = [vp, C.POINTER(StepArgs), C.POINTER(HostOut)]
    lib.d2c_commit.argtypes = [vp, i32, i32, vp, vp, vp, vp, vp, i32, f32]
    lib.d2c_state_ptrs.argtypes = [vp, C.POINTER(State)]
    lib.d2c_sync_status.argtypes = [vp]
    lib.d2c_last_error.restype = C.c_char_p
    lib.d2c_last_error.argtypes = [vp]
    lib.d2c_destroy.argtypes = [vp]
    lib.d2c_profile.argtypes = [vp, i32]
    lib.d2c_profile_read.argtypes = [vp, C.POINTER(C.c_float), C.POINTER(C.c_int64), i32]
    lib.d2c_phase_name.restype = C.c_char_p
    lib.d2c_phase_name.argtypes = [i32]
    lib.d2c_op_select_scratch_bytes.restype = sz
    lib.d2c_op_select_scratch_bytes.argtypes = [i32, i32]
    lib.d2c_op_select.argtypes = [vp, vp, vp, vp, vp, vp, i32, i32, i32, f32, f32, i32, vp, vp, vp, vp, vp, vp, vp, sz, vp]
    lib.d2c_op_gemm.argtypes = [vp, vp, vp, vp, vp, i32, i32, i32, i32, vp]
    lib.d2c_op_attention.argtypes = [vp, i32, i32, vp, vp, vp, i32, i32, i32, i32, i32, i32, vp, vp, vp, i32, vp]
    lib.d2c_op_lm_head_scratch_bytes.restype = sz
    lib.d2c_op_lm_head_scratch_bytes.argtypes = [i32, i32]
    lib.d2c_op_lm_head.argtypes = [vp, vp, vp, i32, i32, i32, vp, vp, vp, vp, sz, vp]
    lib.d2c_op_rollout_scratch_bytes.restype = sz
    lib.d2c_op_rollout_scratch_bytes.argtypes = [i32, i32]
    lib.d2c_op_rollout.argtypes = [vp, sz, i32, vp, vp, i32, i32, vp, vp, sz, vp]
    lib.d2c_op_rollout_static.argtypes = [vp, sz, i32, vp, vp, i32, i32, vp, vp]
    for name in SYMBOLS:
        fn = getattr(lib, name)
        if fn.restype is C.c_int:
            fn.restype = C.c_int
    _lib = lib
    return lib


def _ptr(t: Optional[torch.Tensor]) -> Optional[int]:
    if t is None:
        return None
    assert t.is_contiguous(), "d2c tensors must be contiguous"
    return t.data_ptr()


def _stream_ptr(stream: Optional[torch.cuda.Stream] = None) -> int:
    s = stream if stream is not None else torch.cuda.current_stream()
    return s.cuda_stream


def last_error(ctx: Optional[int] = None) -> str:
    return load().d2c_last_error(ctx).decode()


def _check(rc: int, ctx: Optional[int] = None) -> None:
    if rc != D2C_OK:
        raise D2cError(rc, last_error(ctx))


def make_config(shape, max_batch: int, max_seq: int, sigma: float = 10.0, stage2_candidates: int = 0,
                rollout_layers: int = 0, flags: int = 0) -> Config:
    return Config(shape.n_layers, shape.d_model, shape.n_q_heads, shape.n_kv_heads, shape.head_dim, shape.d_ffn,
                  shape.vocab, max_batch, max_seq, shape.rope_base, shape.rms_eps, sigma, int(shape.qkv_bias),
                  stage2_candidates, rollout_layers, flags)


def d2c_workspace_bytes(cfg: Config) -> int:
    return int(load().d2c_workspace_bytes(C.byref(cfg)))


class Context:
    """Owns the workspace tensor and the handle; methods mirror the C entry points."""

    def __init__(self, cfg: Config, weights: Dict[str, object], device: str = "cuda",
                 stream: Optional[torch.cuda.Stream] = None):
        lib = load()
        self.cfg = cfg
        self.weights = weights                      # keep the borrowed tensors alive
        need = d2c_workspace_bytes(cfg)
        if need == 0:
            raise D2cError(D2C_ESHAPE, "unsupported configuration")
        self.workspace = torch.empty(need + 256, dtype=torch.uint8, device=device)
        base = (self.workspace.data_ptr() + 255) // 256 * 256
        n = cfg.n_layers
        self._arrays = {}
        w = Weights()
        for name in ("wqkv", "bqkv", "wo", "w_gate", "w_up", "w_down", "g_attn", "g_ffn"):
            vals = [lyr[name] for lyr in weights["layers"]]
            if name == "bqkv" and any(v is None for v in vals):
                setattr(w, name, None)
                continue
            arr = (C.c_void_p * n)(*[_ptr(v) for v in vals])
            self._arrays[name] = arr
            setattr(w, name, C.cast(arr, C.POINTER(C.c_void_p)))
        w.g_final = _ptr(weights["g_final"])
        w.w_lm = _ptr(weights["w_lm"])
        self.stream = stream
        handle = C.c_void_p()
        _check(lib.d2c_create(C.byref(cfg), C.byref(w), base, need, _stream_ptr(stream), C.byref(handle)))
        self.handle = handle.value
        st = State()
        _check(lib.d2c_state_ptrs(self.handle, C.byref(st)), self.handle)
        self.state = st
        self._base = base

    # -- views into the workspace (no copies) ------------------------------------------------
    def _view(self, ptr: int, numel: int, dtype: torch.dtype) -> torch.Tensor:
        off = int(ptr) - self.workspace.data_ptr()
        nbytes = int(numel) * torch.empty(0, dtype=dtype).element_size()
        return self.workspace[off: off + nbytes].view(dtype)

    def view(self, name: str, batch: Optional[int] = None, seq_len: Optional[int] = None) -> torch.Tensor:
        c = self.cfg
        B = batch or c.max_batch
        L = seq_len or c.max_seq
        R = c.max_batch * c.max_seq
        kv = c.n_kv_heads * c.head_dim
        if name in ("kcache", "vcache"):
            return self._view(getattr(self.state, name), c.n_layers * R * kv, torch.bfloat16).view(
                c.n_layers, c.max_batch, c.max_seq, c.n_kv_heads, c.head_dim)
        if name in ("conf", "c", "key"):
            return self._view(getattr(self.state, name), B * L, torch.float32).view(B, L)
        if name == "pred":
            return self._view(self.state.pred, B * L, torch.int32).view(B, L)
        if name in ("sel_idx", "lm_rows"):
            return self._view(getattr(self.state, name), R, torch.int32)
        if name in ("row_off", "lm_off"):
            return self._view(getattr(self.state, name), B + 1, torch.int32)
        if name == "lse":
            return self._view(self.state.lse, R * c.n_q_heads, torch.float32).view(R, c.n_q_heads)
        if name == "status":
            return self._view(self.state.status, 4, torch.int32)
        if name == "gemm_clocks":
            return self._view(self.state.gemm_clocks, 4, torch.int64)
        raise KeyError(name)

    def abar(self, layer: int, n_rows: int, seq_len: int) -> torch.Tensor:
        c = self.cfg
        n_rows, seq_len = int(n_rows), int(seq_len)
        stride = c.max_batch * c.max_seq * c.max_seq
        ptr = self.state.abar + int(layer) * stride * 4
        return self._view(ptr, n_rows * seq_len, torch.float32).view(n_rows, seq_len)

    # -- entry points ---------------------------------------------------------------------------
    def step(self, h0: torch.Tensor, mask: torch.Tensor, k: int, p: float, forced: Optional[torch.Tensor] = None,
             forced_off: Optional[torch.Tensor] = None, override_key: Optional[torch.Tensor] = None,
             override_c: Optional[torch.Tensor] = None, hidden_out: Optional[torch.Tensor] = None,
             sel_idx: Optional[torch.Tensor] = None, row_off: Optional[torch.Tensor] = None,
             logits: Optional[torch.Tensor] = None, layer_in: Optional[torch.Tensor] = None,
             block: Optional[Sequence[int]] = None) -> None:
        B, L = mask.shape
        lo, hi = (int(block[0]), int(block[1])) if block is not None else (0, 0)
        a = StepArgs(B, L, _ptr(h0), _ptr(mask), _ptr(forced), _ptr(forced_off), int(k), float(p),
                     _ptr(override_key), _ptr(override_c), lo, hi)
        o = StepOut(_ptr(sel_idx), _ptr(row_off), _ptr(hidden_out), _ptr(logits), _ptr(layer_in))
        _check(load().d2c_step(self.handle, C.byref(a), C.byref(o)), self.handle)

    def step_host(self, h0: torch.Tensor, mask: torch.Tensor, k: int, p: float, forced=None, forced_off=None,
                  override_key=None, override_c=None, sel_idx=None, row_off=None, hidden_out=None, conf=None,
                  pred=None) -> None:
        for t in (h0, mask, forced, forced_off, override_key, override_c, sel_idx, row_off, hidden_out, conf, pred):
            assert t is None or not t.is_cuda, "step_host takes host tensors"
        B, L = mask.shape
        a = StepArgs(B, L, _ptr(h0), _ptr(mask), _ptr(forced), _ptr(forced_off), int(k), float(p),
                     _ptr(override_key), _ptr(override_c), 0, 0)
        o = HostOut(_ptr(sel_idx), _ptr(row_off), _ptr(hidden_out), _ptr(conf), _ptr(pred))
        _check(load().d2c_step_host(self.handle, C.byref(a), C.byref(o)), self.handle)

    def commit(self, embed: torch.Tensor, h0: torch.Tensor, mask: torch.Tensor, tokens: torch.Tensor,
               committed: torch.Tensor, rule: int = 0, threshold: float = 0.9) -> None:
        B, L = mask.shape
        _check(load().d2c_commit(self.handle, B, L, _ptr(embed), _ptr(h0), _ptr(mask), _ptr(tokens), _ptr(committed),
                                 int(rule), float(threshold)), self.handle)

    def profile(self, enable: bool) -> None:
        _check(load().d2c_profile(self.handle, int(enable)), self.handle)

    def profile_read(self, reset: bool = True) -> Dict[str, Dict[str, float]]:
        lib = load()
        ms = (C.c_float * N_PHASES)()
        ln = (C.c_int64 * N_PHASES)()
        _check(lib.d2c_profile_read(self.handle, ms, ln, int(reset)), self.handle)
        return {lib.d2c_phase_name(i).decode(): {"ms": float(ms[i]), "launches": int(ln[i])} for i in range(N_PHASES)}

    def sync_status(self) -> None:
        _check(load().d2c_sync_status(self.handle), self.handle)

    def close(self) -> None:
        if getattr(self, "handle", None):
            load().d2c_destroy(self.handle)
            self.handle = None

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass


# -- stand-alone kernels ----------------------------------------------------------------------------
def _scratch(nbytes: int, device) -> torch.Tensor:
    t = torch.empty(nbytes + 256, dtype=torch.uint8, device=device)
    off = (-t.data_ptr()) % 256
    return t[off: off + nbytes]


def d2c_op_select(mask, conf, c, k, p, sigma=10.0, stage2_candidates=0, override_key=None, forced=None,
                  forced_off=None):
    lib = load()
    B, L = mask.shape
    dev = mask.device
    key = torch.empty(B, L, dtype=torch.float32, device=dev)
    sel_idx = torch.full((B * L,), -1, dtype=torch.int32, device=dev)
    row_off = torch.zeros(B + 1, dtype=torch.int32, device=dev)
    lm_rows = torch.full((B * L,), -1, dtype=torch.int32, device=dev)
    lm_off = torch.zeros(B + 1, dtype=torch.int32, device=dev)
    slot = torch.empty(B, L, dtype=torch.int32, device=dev)
    nb = int(lib.d2c_op_select_scratch_bytes(B, L))
    scratch = _scratch(nb, dev)
    _check(lib.d2c_op_select(_ptr(mask), _ptr(conf), _ptr(c), _ptr(override_key), _ptr(forced), _ptr(forced_off), B, L,
                             int(k), float(p), float(sigma), int(stage2_candidates), _ptr(key), _ptr(sel_idx),
                             _ptr(row_off), _ptr(lm_rows), _ptr(lm_off), _ptr(slot), scratch.data_ptr(), nb,
                             _stream_ptr()))
    return dict(key=key, sel_idx=sel_idx, row_off=row_off, lm_rows=lm_rows, lm_off=lm_off, slot_of_pos=slot)


def d2c_op_gemm(A, W, n_rows, bias=None, impl=0):
    max_rows, K = A.shape
    N = W.shape[0]
    Cm = torch.zeros(max_rows, N, dtype=torch.bfloat16, device=A.device)
    _check(load().d2c_op_gemm(_ptr(A), _ptr(W), _ptr(bias), _ptr(Cm), _ptr(n_rows), max_rows, N, K, int(impl),
                              _stream_ptr()))
    return Cm


def d2c_op_attention(q, kcache, vcache, row_off, seq_len, n_q_heads, n_kv_heads, head_dim, want_abar=True, impl=0):
    rows, ldq = q.shape
    B, cache_seq = kcache.shape[0], kcache.shape[1]
    dev = q.device
    o = torch.zeros(rows, n_q_heads * head_dim, dtype=torch.bfloat16, device=dev)
    lse = torch.zeros(rows, n_q_heads, dtype=torch.float32, device=dev)
    abar = torch.zeros(rows, seq_len, dtype=torch.float32, device=dev) if want_abar else None
    _check(load().d2c_op_attention(_ptr(q), rows, ldq, _ptr(kcache), _ptr(vcache), _ptr(row_off), B, seq_len, cache_seq,
                                   n_q_heads, n_kv_heads, head_dim, _ptr(o), _ptr(lse), _ptr(abar), int(impl), _stream_ptr()))
    return o, lse, abar


def d2c_op_lm_head(x, w_lm, n_rows, want_logits=False):
    lib = load()
    max_rows, d = x.shape
    V = w_lm.shape[0]
    dev = x.device
    conf = torch.zeros(max_rows, dtype=torch.float32, device=dev)
    pred = torch.full((max_rows,), -1, dtype=torch.int32, device=dev)
    logits = torch.zeros(max_rows, V, dtype=torch.float32, device=dev) if want_logits else None
    nb = int(lib.d2c_op_lm_head_scratch_bytes(max_rows, V))
    scratch = _scratch(nb, dev)
    _check(lib.d2c_op_lm_head(_ptr(x), _ptr(w_lm), _ptr(n_rows), max_rows, d, V, _ptr(conf), _ptr(pred), _ptr(logits),
                              scratch.data_ptr(), nb, _stream_ptr()))
    return conf, pred, logits


def d2c_op_rollout(abar, sel_idx, row_off, batch, seq_len, c=None):
    lib = load()
    n_layers = abar.shape[0]
    layer_stride = abar.stride(0)
    dev = abar.device
    if c is None:
        c = torch.zeros(batch, seq_len, dtype=torch.float32, device=dev)
    nb = int(lib.d2c_op_rollout_scratch_bytes(batch, seq_len))
    scratch = _scratch(nb, dev)
    _check(lib.d2c_op_rollout(_ptr(abar), layer_stride, n_layers, _ptr(sel_idx), _ptr(row_off), batch, seq_len,
                              _ptr(c), scratch.data_ptr(), nb, _stream_ptr()))
    return c


def d2c_op_rollout_static(abar, sel_idx, row_off, batch, seq_len, c=None):
    """d2c_op_rollout for callers that cannot allocate: the scratch is a fixed array inside the library
    (batch * seq_len <= 16384).  This wrapper itself only creates the output tensor when none is given."""
    if c is None:
        c = torch.zeros(batch, seq_len, dtype=torch.float32, device=abar.device)
    _check(load().d2c_op_rollout_static(_ptr(abar), abar.stride(0), abar.shape[0], _ptr(sel_idx), _ptr(row_off), batch,
                                        seq_len, _ptr(c), _stream_ptr()))
    return c


def d2c_op_wait_probe(status: torch.Tensor, limit_cycles: int = 100000):
    """Runs the library's bounded device-side wait on a barrier nothing arrives on; status: int32[4] on the device."""
    assert status.dtype == torch.int32 and status.numel() >= 4
    lib = load()
    lib.d2c_op_wait_probe.argtypes = [C.c_void_p, C.c_int64, C.c_void_p]
    _check(lib.d2c_op_wait_probe(_ptr(status), int(limit_cycles), _stream_ptr()))
