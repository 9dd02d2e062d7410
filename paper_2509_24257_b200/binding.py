"""Thin ctypes binding over the C ABI of libverillm.so (include/verillm.h).

Argument marshalling only: torch supplies device memory and the stream, every step of the path
runs in the library's kernels.  There is no CPU fallback: a missing library raises on first use.
"""
from __future__ import annotations

import ctypes as C
import os
from typing import Dict, List, Optional, Sequence

import numpy as np
import torch

_HERE = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(_HERE, "libverillm.so")

NSTAT = 16
STAT_NAMES = (
    "rel_l2", "max_abs", "mae", "mean_signed", "p_e", "p_m", "p_w", "q_small", "z_large",
    "n_exp_mismatch", "n_mant_large", "n_mant_small", "n_exact", "n_nonfinite", "l2_delta", "l2_ref",
)
BF16, F32 = 0, 1
TOL_BIT_AWARE = 1
E_INVAL, E_SHAPE, E_RANGE, E_NOMEM, E_CUDA, E_ARCH = -1, -2, -3, -4, -5, -6
DEV_TOKEN_RANGE, DEV_WAIT_TIMEOUT = 1, 2

EXPORTS = (
    "verillm_default_tol", "verillm_load_weights", "verillm_load_layer", "verillm_load_globals",
    "verillm_verify_prefill", "verillm_decode_commit", "verillm_compare", "verillm_compare_noalloc", "verillm_op_gemm",
    "verillm_op_rmsnorm", "verillm_op_attention", "verillm_free", "verillm_strerror",
    "verillm_last_launch_count", "verillm_profile_enable", "verillm_profile_read",
    "verillm_load_lm_head", "verillm_token_match", "verillm_verify_segment", "verillm_spot_check", "verillm_merkle_roots",
    "verillm_threshold_sweep", "verillm_selftest_wait_timeout",
)
PROF_CLASSES = ("setup", "rmsnorm", "gemm_qkv_rope", "attention", "gemm_o_resid", "gemm_gate_up_swiglu",
                "gemm_down_resid_compare", "verdict")


class VerillmError(RuntimeError):
    def __init__(self, code: int, what: str):
        super().__init__(f"{what}: error {code} ({strerror(code)})")
        self.code = code


class Config(C.Structure):
    _fields_ = [(n, C.c_int32) for n in ("n_layers", "d_model", "n_heads", "n_kv_heads", "head_dim", "d_ffn", "vocab")] + [
        ("rope_base", C.c_float), ("rms_eps", C.c_float),
        ("max_tokens", C.c_int32), ("max_checks", C.c_int32), ("max_batch", C.c_int32),
    ]


class LayerWeights(C.Structure):
    _fields_ = [(n, C.c_void_p) for n in ("attn_norm", "wq", "wk", "wv", "wo", "ffn_norm", "w_gate", "w_up", "w_down")]


class Weights(C.Structure):
    _fields_ = [("embed", C.c_void_p), ("final_norm", C.c_void_p), ("layers", C.POINTER(LayerWeights)), ("on_device", C.c_int32)]


class Tol(C.Structure):
    _fields_ = [
        ("rel_l2", C.c_float), ("max_abs", C.c_float), ("mae", C.c_float),
        ("pe_max", C.c_float), ("pm_min", C.c_float), ("pw_min", C.c_float), ("e_abs_max", C.c_float),
        ("e_w", C.c_float), ("e_m", C.c_int32),
        ("tau_large", C.c_float), ("z_large_max", C.c_float), ("q_small_min", C.c_float),
        ("flags", C.c_uint32),
    ]


class ReportC(C.Structure):
    _fields_ = [(n, C.c_void_p) for n in ("stats", "pos_ok", "first_bad_layer", "seq_ok", "seq_score", "hidden_out", "status")]


_lib: Optional[C.CDLL] = None


def lib() -> C.CDLL:
    """Loads libverillm.so (built in-tree by paper_2509_24257_b200.build); raises if it is missing."""
    global _lib
    if _lib is None:
        if not os.path.exists(LIB_PATH):
            raise FileNotFoundError(
                f"{LIB_PATH} is missing: build it with `python -m paper_2509_24257_b200.build` "
                "(there is no fallback implementation)"
            )
        L = C.CDLL(LIB_PATH)
        L.verillm_strerror.restype = C.c_char_p
        L.verillm_strerror.argtypes = [C.c_int]
        L.verillm_default_tol.restype = None
        L.verillm_default_tol.argtypes = [C.POINTER(Tol)]
        L.verillm_free.restype = None
        L.verillm_free.argtypes = [C.c_void_p]
        L.verillm_last_launch_count.restype = C.c_int32
        L.verillm_last_launch_count.argtypes = [C.c_void_p]
        L.verillm_load_weights.argtypes = [C.POINTER(Config), C.POINTER(Weights), C.POINTER(C.c_void_p)]
        L.verillm_load_layer.argtypes = [C.c_void_p, C.c_int32, C.POINTER(LayerWeights), C.c_int32]
        L.verillm_load_globals.argtypes = [C.c_void_p, C.c_void_p, C.c_void_p, C.c_int32]
        L.verillm_verify_prefill.argtypes = [
            C.c_void_p, C.c_void_p, C.c_void_p, C.c_int32, C.c_void_p, C.c_int32, C.c_void_p, C.c_void_p, C.c_int32,
            C.POINTER(Tol), C.POINTER(ReportC), C.c_void_p,
        ]
        L.verillm_decode_commit.argtypes = [
            C.c_void_p, C.c_void_p, C.c_void_p, C.c_int32, C.c_int32, C.c_void_p, C.c_void_p, C.c_int32, C.c_void_p,
            C.c_int32, C.c_void_p, C.c_void_p,
        ]
        L.verillm_compare.argtypes = [
            C.c_void_p, C.c_void_p, C.c_int32, C.c_int32, C.c_int32, C.c_int32, C.c_void_p, C.c_int32,
            C.POINTER(Tol), C.POINTER(ReportC), C.c_void_p,
        ]
        L.verillm_compare_noalloc.argtypes = L.verillm_compare.argtypes
        L.verillm_compare_noalloc.restype = C.c_int
        L.verillm_verify_segment.argtypes = [
            C.c_void_p, C.c_void_p, C.c_int32, C.c_int32, C.c_int32, C.c_void_p, C.c_int32, C.c_void_p, C.c_int32,
            C.c_void_p, C.c_void_p, C.c_int32, C.POINTER(Tol), C.POINTER(ReportC), C.c_void_p,
        ]
        L.verillm_verify_segment.restype = C.c_int
        L.verillm_spot_check.argtypes = [C.c_void_p, C.c_int32, C.c_int32, C.c_void_p, C.c_void_p, C.c_void_p, C.c_int32,
                                         C.c_float, C.c_float, C.c_void_p, C.c_void_p, C.c_void_p, C.c_void_p]
        L.verillm_spot_check.restype = C.c_int
        L.verillm_merkle_roots.argtypes = [C.c_void_p, C.c_int32, C.c_int32, C.c_void_p, C.c_void_p]
        L.verillm_merkle_roots.restype = C.c_int
        L.verillm_threshold_sweep.argtypes = [C.c_void_p, C.c_void_p, C.c_int32, C.POINTER(Tol), C.c_int32, C.c_void_p, C.c_void_p]
        L.verillm_threshold_sweep.restype = C.c_int
        L.verillm_selftest_wait_timeout.argtypes = [C.c_int64, C.c_void_p, C.c_void_p, C.c_void_p]
        L.verillm_selftest_wait_timeout.restype = C.c_int
        L.verillm_load_lm_head.argtypes = [C.c_void_p, C.c_void_p, C.c_int32]
        L.verillm_load_lm_head.restype = C.c_int
        L.verillm_token_match.argtypes = [C.c_void_p, C.c_void_p, C.c_void_p, C.c_int32, C.c_void_p, C.c_void_p, C.c_void_p, C.c_void_p]
        L.verillm_token_match.restype = C.c_int
        L.verillm_op_gemm.argtypes = [C.c_void_p, C.c_void_p, C.c_void_p, C.c_int32, C.c_int32, C.c_int32, C.c_int32, C.c_void_p, C.c_void_p]
        L.verillm_op_rmsnorm.argtypes = [C.c_void_p, C.c_void_p, C.c_void_p, C.c_int32, C.c_int32, C.c_float, C.c_void_p]
        L.verillm_op_attention.argtypes = [C.c_void_p, C.c_void_p, C.c_int32, C.c_int32, C.c_int32, C.c_int32, C.c_int32, C.c_int32, C.c_void_p, C.c_void_p]
        L.verillm_profile_enable.argtypes = [C.c_void_p, C.c_int32]
        L.verillm_profile_read.argtypes = [C.c_void_p, C.POINTER(C.c_float), C.POINTER(C.c_int32)]
        L.verillm_profile_enable.restype = C.c_int
        L.verillm_profile_read.restype = C.c_int
        for name in ("verillm_load_weights", "verillm_load_layer", "verillm_load_globals", "verillm_verify_prefill",
                     "verillm_decode_commit", "verillm_compare", "verillm_compare_noalloc", "verillm_op_gemm", "verillm_op_rmsnorm",
                     "verillm_op_attention"):
            getattr(L, name).restype = C.c_int
        _lib = L
    return _lib


def strerror(code: int) -> str:
    return lib().verillm_strerror(code).decode()


def _check(code: int, what: str) -> None:
    if code != 0:
        raise VerillmError(code, what)


def default_tol(**overrides) -> Tol:
    t = Tol()
    lib().verillm_default_tol(C.byref(t))
    for k, v in overrides.items():
        if k == "bit_aware":
            t.flags = (t.flags | TOL_BIT_AWARE) if v else (t.flags & ~TOL_BIT_AWARE)
        else:
            setattr(t, k, v)
    return t


def _stream_ptr(stream: Optional[torch.cuda.Stream]) -> int:
    return (stream or torch.cuda.current_stream()).cuda_stream


def _i32(a) -> np.ndarray:
    return np.ascontiguousarray(np.asarray(a, dtype=np.int32))


def _ptr(t: Optional[torch.Tensor]) -> Optional[int]:
    return None if t is None else t.data_ptr()


class Report:
    """Device tensors of one verification report; `.cpu()` copies them into numpy arrays."""

    def __init__(self, n_check: int, n_layers: int, batch: int, d_model: int, device, want_hidden: bool):
        nc = max(n_check, 1)
        self.n_check, self.n_layers, self.batch = n_check, n_layers, batch
        self.stats = torch.zeros(nc, n_layers, NSTAT, dtype=torch.float32, device=device)
        self.pos_ok = torch.zeros(nc, dtype=torch.uint8, device=device)
        self.first_bad_layer = torch.zeros(nc, dtype=torch.int32, device=device)
        self.seq_ok = torch.zeros(batch, dtype=torch.uint8, device=device)
        self.seq_score = torch.zeros(batch, dtype=torch.float32, device=device)
        self.hidden = torch.zeros(n_layers, nc, d_model, dtype=torch.float32, device=device) if want_hidden else None
        self.status = torch.zeros(1, dtype=torch.int32, device=device)

    def c_struct(self) -> ReportC:
        return ReportC(_ptr(self.stats), _ptr(self.pos_ok), _ptr(self.first_bad_layer), _ptr(self.seq_ok),
                       _ptr(self.seq_score), _ptr(self.hidden), _ptr(self.status))

    def cpu(self) -> Dict[str, np.ndarray]:
        n = self.n_check
        out = {
            "stats": self.stats[:n].cpu().numpy(), "pos_ok": self.pos_ok[:n].cpu().numpy(),
            "first_bad_layer": self.first_bad_layer[:n].cpu().numpy(), "seq_ok": self.seq_ok.cpu().numpy(),
            "seq_score": self.seq_score.cpu().numpy(), "status": int(self.status.item()),
        }
        if self.hidden is not None:
            out["hidden"] = self.hidden[:, :n].cpu().numpy()
        return out


_LAYER_KEYS = ("attn_norm", "wq", "wk", "wv", "wo", "ffn_norm", "w_gate", "w_up", "w_down")


def _layer_struct(lw: Dict[str, torch.Tensor]) -> LayerWeights:
    for k in _LAYER_KEYS:
        t = lw[k]
        if t.dtype != torch.bfloat16 or not t.is_contiguous():
            raise ValueError(f"layer tensor {k} must be contiguous bf16")
    return LayerWeights(*[lw[k].data_ptr() for k in _LAYER_KEYS])


class Model:
    """Handle on the library's copy of a model (verillm_load_weights / verillm_free)."""

    def __init__(self, shape, max_tokens: int, max_checks: int, max_batch: int, device: str | torch.device = "cuda:0"):
        self.shape = shape
        self.device = torch.device(device)
        self.cfg = Config(shape.n_layers, shape.d_model, shape.n_heads, shape.n_kv_heads, shape.head_dim, shape.d_ffn,
                          shape.vocab, float(shape.rope_base), float(shape.rms_eps), max_tokens, max_checks, max_batch)
        self._h = C.c_void_p()
        with torch.cuda.device(self.device):
            _check(lib().verillm_load_weights(C.byref(self.cfg), None, C.byref(self._h)), "verillm_load_weights")

    @classmethod
    def from_weights(cls, shape, weights: Dict[str, object], max_tokens: int, max_checks: int, max_batch: int,
                     device: str | torch.device = "cuda:0") -> "Model":
        m = cls(shape, max_tokens, max_checks, max_batch, device)
        m.load_globals(weights["embed"], weights["final_norm"])
        for l, lw in enumerate(weights["layers"]):
            m.load_layer(l, lw)
        return m

    def load_globals(self, embed: torch.Tensor, final_norm: torch.Tensor) -> None:
        on_dev = int(embed.is_cuda)
        with torch.cuda.device(self.device):
            _check(lib().verillm_load_globals(self._h, embed.data_ptr(), final_norm.data_ptr(), on_dev), "verillm_load_globals")

    def load_layer(self, layer: int, lw: Dict[str, torch.Tensor]) -> None:
        on_dev = int(lw["wq"].is_cuda)
        st = _layer_struct(lw)
        with torch.cuda.device(self.device):
            _check(lib().verillm_load_layer(self._h, layer, C.byref(st), on_dev), "verillm_load_layer")

    def verify_prefill(self, tokens: torch.Tensor, cu_seqlens: Sequence[int], committed: Optional[torch.Tensor],
                       check_seq: Sequence[int], check_pos: Sequence[int], tol: Optional[Tol] = None,
                       want_hidden: bool = False, report: Optional[Report] = None,
                       stream: Optional[torch.cuda.Stream] = None) -> Report:
        """tokens: int32 device [n_tokens]; committed: device [n_layers][n_check][d_model] bf16 or f32."""
        cu = _i32(cu_seqlens)
        cs, cp = _i32(check_seq), _i32(check_pos)
        n_check, batch = int(cs.shape[0]), int(cu.shape[0]) - 1
        tol = tol or default_tol()
        if report is None:
            report = Report(n_check, self.shape.n_layers, batch, self.shape.d_model, self.device, want_hidden)
        dtype = BF16
        if committed is not None:
            if committed.dtype == torch.float32:
                dtype = F32
            elif committed.dtype != torch.bfloat16:
                raise ValueError("committed states must be bf16 or float32")
            if not committed.is_contiguous():
                raise ValueError("committed states must be contiguous")
        if tokens.dtype != torch.int32 or not tokens.is_cuda:
            raise ValueError("tokens must be an int32 CUDA tensor")
        rc_struct = report.c_struct()
        with torch.cuda.device(self.device):
            code = lib().verillm_verify_prefill(
                self._h, tokens.data_ptr(), cu.ctypes.data, batch, _ptr(committed), dtype, cs.ctypes.data, cp.ctypes.data,
                n_check, C.byref(tol), C.byref(rc_struct), _stream_ptr(stream))
        _check(code, "verillm_verify_prefill")
        return report

    def verify_segment(self, input_states: torch.Tensor, layer_begin: int, layer_end: int, cu_seqlens: Sequence[int],
                       committed: Optional[torch.Tensor], check_seq: Sequence[int], check_pos: Sequence[int],
                       tol: Optional[Tol] = None, want_hidden: bool = False,
                       stream: Optional[torch.cuda.Stream] = None) -> Report:
        """input_states: device [n_tokens][d_model] bf16/f32; committed: device [layer_end-layer_begin][n_check][d_model]."""
        cu = _i32(cu_seqlens)
        cs, cp = _i32(check_seq), _i32(check_pos)
        n_check, batch = int(cs.shape[0]), int(cu.shape[0]) - 1
        tol = tol or default_tol()
        report = Report(n_check, layer_end - layer_begin, batch, self.shape.d_model, self.device, want_hidden)
        if not input_states.is_contiguous() or input_states.dtype not in (torch.bfloat16, torch.float32):
            raise ValueError("input states must be contiguous bf16 or float32")
        cdt = BF16 if committed is None or committed.dtype == torch.bfloat16 else F32
        st = report.c_struct()
        with torch.cuda.device(self.device):
            code = lib().verillm_verify_segment(
                self._h, input_states.data_ptr(), BF16 if input_states.dtype == torch.bfloat16 else F32, layer_begin,
                layer_end, cu.ctypes.data, batch, _ptr(committed), cdt, cs.ctypes.data, cp.ctypes.data, n_check,
                C.byref(tol), C.byref(st), _stream_ptr(stream))
        _check(code, "verillm_verify_segment")
        return report

    def decode_commit(self, tokens: torch.Tensor, cu_seqlens: Sequence[int], n_prefill: int, check_seq: Sequence[int],
                      check_pos: Sequence[int], commit_dtype: torch.dtype = torch.bfloat16,
                      stream: Optional[torch.cuda.Stream] = None) -> torch.Tensor:
        cu = _i32(cu_seqlens)
        cs, cp = _i32(check_seq), _i32(check_pos)
        n_check, batch = int(cs.shape[0]), int(cu.shape[0]) - 1
        out = torch.zeros(self.shape.n_layers, max(n_check, 1), self.shape.d_model, dtype=commit_dtype, device=self.device)
        status = torch.zeros(1, dtype=torch.int32, device=self.device)
        with torch.cuda.device(self.device):
            code = lib().verillm_decode_commit(
                self._h, tokens.data_ptr(), cu.ctypes.data, batch, int(n_prefill), cs.ctypes.data, cp.ctypes.data, n_check,
                out.data_ptr(), BF16 if commit_dtype == torch.bfloat16 else F32, status.data_ptr(), _stream_ptr(stream))
        _check(code, "verillm_decode_commit")
        if int(status.item()) != 0:
            raise RuntimeError(f"verillm_decode_commit: device status {int(status.item())}")
        return out[:, :n_check]

    def load_lm_head(self, lm_head: torch.Tensor) -> None:
        if lm_head.dtype != torch.bfloat16 or not lm_head.is_contiguous():
            raise ValueError("the output head must be contiguous bf16")
        with torch.cuda.device(self.device):
            _check(lib().verillm_load_lm_head(self._h, lm_head.data_ptr(), int(lm_head.is_cuda)), "verillm_load_lm_head")

    def token_match(self, last_hidden: torch.Tensor, claimed: Sequence[int], stream: Optional[torch.cuda.Stream] = None):
        """last_hidden: float32 device [n_check][d_model].  Returns device tensors (argmax int32, match uint8, margin f32)."""
        cl = _i32(claimed)
        n = int(cl.shape[0])
        if last_hidden.dtype != torch.float32 or not last_hidden.is_contiguous() or last_hidden.shape[0] != n:
            raise ValueError("last_hidden must be contiguous float32 [n_check][d_model]")
        arg = torch.empty(n, dtype=torch.int32, device=self.device)
        match = torch.empty(n, dtype=torch.uint8, device=self.device)
        margin = torch.empty(n, dtype=torch.float32, device=self.device)
        with torch.cuda.device(self.device):
            _check(lib().verillm_token_match(self._h, last_hidden.data_ptr(), cl.ctypes.data, n, arg.data_ptr(),
                                             match.data_ptr(), margin.data_ptr(), _stream_ptr(stream)), "verillm_token_match")
        return arg, match, margin

    def profile_enable(self, on: bool = True) -> None:
        with torch.cuda.device(self.device):
            _check(lib().verillm_profile_enable(self._h, int(on)), "verillm_profile_enable")

    def profile_read(self) -> Dict[str, tuple]:
        """{kernel class: (milliseconds, launches)} of the last verify_prefill call."""
        ms = (C.c_float * len(PROF_CLASSES))()
        n = (C.c_int32 * len(PROF_CLASSES))()
        with torch.cuda.device(self.device):
            _check(lib().verillm_profile_read(self._h, ms, n), "verillm_profile_read")
        return {k: (float(ms[i]), int(n[i])) for i, k in enumerate(PROF_CLASSES)}

    def last_launch_count(self) -> int:
        return int(lib().verillm_last_launch_count(self._h))

    def close(self) -> None:
        if self._h:
            with torch.cuda.device(self.device):
                lib().verillm_free(self._h)
            self._h = C.c_void_p()

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass


def compare(hidden: torch.Tensor, committed: torch.Tensor, check_seq: Sequence[int], batch: int,
            tol: Optional[Tol] = None, stream: Optional[torch.cuda.Stream] = None) -> Report:
    """Comparison and verdict on given states: hidden f32 [L][n][d], committed bf16/f32 [L][n][d] (device)."""
    n_layers, n_check, d = hidden.shape
    cs = _i32(check_seq)
    tol = tol or default_tol()
    rep = Report(n_check, n_layers, batch, d, hidden.device, False)
    st = rep.c_struct()
    with torch.cuda.device(hidden.device):
        code = lib().verillm_compare(hidden.data_ptr(), committed.data_ptr(), BF16 if committed.dtype == torch.bfloat16 else F32,
                                     n_layers, n_check, d, cs.ctypes.data, batch, C.byref(tol), C.byref(st), _stream_ptr(stream))
    _check(code, "verillm_compare")
    return rep


def compare_noalloc(hidden: torch.Tensor, committed: torch.Tensor, check_seq: Sequence[int], batch: int,
                    tol: Optional[Tol] = None, report: Optional[Report] = None,
                    stream: Optional[torch.cuda.Stream] = None) -> Report:
    """verillm_compare_noalloc: like `compare`, but the library's scratch is a fixed array inside the library,
    so the call itself allocates nothing.  Pass a `report` made beforehand to keep this wrapper from
    allocating the output tensors too.  Raises E_SHAPE beyond n_layers * n_check = 65536."""
    n_layers, n_check, d = hidden.shape
    cs = _i32(check_seq)
    tol = tol or default_tol()
    rep = report or Report(n_check, n_layers, batch, d, hidden.device, False)
    st = rep.c_struct()
    with torch.cuda.device(hidden.device):
        code = lib().verillm_compare_noalloc(hidden.data_ptr(), committed.data_ptr(),
                                             BF16 if committed.dtype == torch.bfloat16 else F32, n_layers, n_check, d,
                                             cs.ctypes.data, batch, C.byref(tol), C.byref(st), _stream_ptr(stream))
    _check(code, "verillm_compare_noalloc")
    return rep


def spot_check(hidden: torch.Tensor, sample_row, sample_col, reference, eps: float, theta: float,
               stream: Optional[torch.cuda.Stream] = None):
    """Sampled value matching on hidden (float32 device [n_rows][d]).  Returns device (agree uint8 [n], p_hat f32 [1], ok uint8 [1])."""
    rows, cols = _i32(sample_row), _i32(sample_col)
    ref = np.ascontiguousarray(np.asarray(reference, dtype=np.float32))
    n = int(rows.shape[0])
    agree = torch.empty(n, dtype=torch.uint8, device=hidden.device)
    p_hat = torch.empty(1, dtype=torch.float32, device=hidden.device)
    ok = torch.empty(1, dtype=torch.uint8, device=hidden.device)
    with torch.cuda.device(hidden.device):
        _check(lib().verillm_spot_check(hidden.data_ptr(), hidden.shape[0], hidden.shape[1], rows.ctypes.data,
                                        cols.ctypes.data, ref.ctypes.data, n, float(eps), float(theta), agree.data_ptr(),
                                        p_hat.data_ptr(), ok.data_ptr(), _stream_ptr(stream)), "verillm_spot_check")
    return agree, p_hat, ok


def threshold_sweep(stats: torch.Tensor, is_attack: torch.Tensor, variants: Sequence[Tol],
                    stream: Optional[torch.cuda.Stream] = None) -> torch.Tensor:
    """stats float32 device [n_cells][NSTAT] (report.stats reshaped), is_attack uint8 device [n_cells], up to 64
    tolerance sets -> int32 device [n_variants][4] = honest accepted, honest rejected, attack accepted, attack rejected."""
    if stats.dtype != torch.float32 or not stats.is_contiguous() or stats.dim() != 2 or stats.shape[1] != NSTAT:
        raise ValueError("stats must be a contiguous float32 [n_cells][NSTAT] tensor")
    if is_attack.dtype != torch.uint8 or not is_attack.is_contiguous() or is_attack.numel() != stats.shape[0]:
        raise ValueError("is_attack must be a contiguous uint8 tensor with one entry per cell")
    arr = (Tol * len(variants))(*variants)
    counts = torch.empty(len(variants), 4, dtype=torch.int32, device=stats.device)
    with torch.cuda.device(stats.device):
        _check(lib().verillm_threshold_sweep(stats.data_ptr(), is_attack.data_ptr(), stats.shape[0], arr, len(variants),
                                             counts.data_ptr(), _stream_ptr(stream)), "verillm_threshold_sweep")
    return counts


def selftest_wait_timeout(limit_cycles: int, device="cuda:0", stream: Optional[torch.cuda.Stream] = None):
    """Runs the library's bounded wait on a barrier nobody signals.  Returns device tensors (status int32 [1],
    gave_up int32 [1])."""
    device = torch.device(device)
    status = torch.zeros(1, dtype=torch.int32, device=device)
    gave_up = torch.zeros(1, dtype=torch.int32, device=device)
    with torch.cuda.device(device):
        _check(lib().verillm_selftest_wait_timeout(int(limit_cycles), status.data_ptr(), gave_up.data_ptr(),
                                                   _stream_ptr(stream)), "verillm_selftest_wait_timeout")
    return status, gave_up


def merkle_roots(states: torch.Tensor, stream: Optional[torch.cuda.Stream] = None,
                 out: Optional[torch.Tensor] = None) -> torch.Tensor:
    """states float32 device [n_vec][d] -> uint8 device [n_vec][32] SHA-256 Merkle roots over float32 leaves
    (written to `out` if given)."""
    if states.dtype != torch.float32 or not states.is_contiguous() or states.dim() != 2:
        raise ValueError("states must be a contiguous float32 matrix")
    roots = out if out is not None else torch.empty(states.shape[0], 32, dtype=torch.uint8, device=states.device)
    if roots.dtype != torch.uint8 or tuple(roots.shape) != (states.shape[0], 32) or not roots.is_contiguous():
        raise ValueError("out must be a contiguous uint8 [n_vec][32] tensor")
    with torch.cuda.device(states.device):
        _check(lib().verillm_merkle_roots(states.data_ptr(), states.shape[0], states.shape[1], roots.data_ptr(),
                                          _stream_ptr(stream)), "verillm_merkle_roots")
    return roots


def op_gemm(a: torch.Tensor, b: torch.Tensor, out_f32: bool = False) -> torch.Tensor:
    """a [M][K] bf16, b [N][K] bf16 -> a @ b.T"""
    M, K = a.shape
    N = b.shape[0]
    c = torch.empty(M, N, dtype=torch.float32 if out_f32 else torch.bfloat16, device=a.device)
    status = torch.zeros(1, dtype=torch.int32, device=a.device)
    with torch.cuda.device(a.device):
        _check(lib().verillm_op_gemm(a.data_ptr(), b.data_ptr(), c.data_ptr(), M, N, K, int(out_f32), status.data_ptr(),
                                     _stream_ptr(None)), "verillm_op_gemm")
    if int(status.item()) != 0:
        raise RuntimeError(f"verillm_op_gemm: device status {int(status.item())}")
    return c


def op_rmsnorm(x: torch.Tensor, gain: torch.Tensor, eps: float) -> torch.Tensor:
    M, d = x.shape
    y = torch.empty(M, d, dtype=torch.bfloat16, device=x.device)
    with torch.cuda.device(x.device):
        _check(lib().verillm_op_rmsnorm(x.data_ptr(), gain.data_ptr(), y.data_ptr(), M, d, float(eps), _stream_ptr(None)),
               "verillm_op_rmsnorm")
    return y


def op_attention(qkv: torch.Tensor, cu_seqlens: Sequence[int], n_heads: int, n_kv_heads: int, head_dim: int) -> torch.Tensor:
    cu = _i32(cu_seqlens)
    M = qkv.shape[0]
    cu_dev = torch.from_numpy(cu).to(qkv.device)
    out = torch.empty(M, n_heads * head_dim, dtype=torch.bfloat16, device=qkv.device)
    max_len = int(np.max(np.diff(cu)))
    with torch.cuda.device(qkv.device):
        _check(lib().verillm_op_attention(qkv.data_ptr(), cu_dev.data_ptr(), len(cu) - 1, max_len, M, n_heads, n_kv_heads,
                                          head_dim, out.data_ptr(), _stream_ptr(None)), "verillm_op_attention")
    return out
