"""Thin ctypes binding of libibert_b200.so: same names as the C ABI (``include/ibert.h``),
argument marshalling only.  Tensors are torch CUDA tensors whose ``data_ptr()`` is passed
through; every step of the computation runs in the library's CUDA kernels.  There is no
CPU path: if the library is missing or a call fails, an exception is raised.
"""
from __future__ import annotations

import ctypes as C
from pathlib import Path

import numpy as np
import torch

_PKG = Path(__file__).resolve().parent
LIB_PATH = _PKG / "libibert_b200.so"
_lib = None

IBERT_OK = 0
ERR_NAMES = {-1: "IBERT_ERR_ARG", -2: "IBERT_ERR_SHAPE", -3: "IBERT_ERR_SCALE_RANGE", -4: "IBERT_ERR_ALIGN",
             -5: "IBERT_ERR_NOMEM", -6: "IBERT_ERR_CUDA", -7: "IBERT_ERR_TIMEOUT", -8: "IBERT_ERR_VALUE_RANGE"}

KERNEL_CLASSES = ("gemm_qkv", "attention", "gemm_out", "layernorm", "gemm_ffn1_gelu", "gemm_ffn2", "gelu",
                  "softmax", "gemm_out_ln", "gemm_ffn2_ln")
SCALE_NAMES = ("S_x", "S_q", "S_k", "S_v", "S_ctx", "S_r1", "S_h1", "S_gi", "S_go", "S_r2", "S_out")


class IbertError(RuntimeError):
    def __init__(self, code: int, where: str):
        msg = lib().ibert_strerror(code).decode() if _lib is not None else "?"
        super().__init__(f"{where}: {ERR_NAMES.get(code, code)} ({msg})")
        self.code = code


class LayerDesc(C.Structure):
    _fields_ = [("H", C.c_int32), ("heads", C.c_int32), ("F", C.c_int32), ("p_max", C.c_int32)] + [
        (n, C.c_void_p) for n in (
            "w_qkv", "S_w_qkv", "bias_qkv", "w_o", "S_w_o", "bias_o",
            "w_f1", "S_w_f1", "bias_f1", "w_f2", "S_w_f2", "bias_f2",
            "gamma1", "beta1", "gamma2", "beta2")] + [(n, C.c_double) for n in SCALE_NAMES]


def lib():
    """Loads the C-ABI library; fails loudly if it has not been built."""
    global _lib
    if _lib is None:
        if not LIB_PATH.exists():
            raise RuntimeError(f"{LIB_PATH} is missing: run `python -m paper_2101_01321_b200.build` "
                               "(there is no fallback path)")
        L = C.CDLL(str(LIB_PATH))
        vp, i32, i64, dbl = C.c_void_p, C.c_int, C.c_int64, C.c_double
        L.ibert_strerror.restype = C.c_char_p
        L.ibert_strerror.argtypes = [i32]
        L.ibert_create.argtypes = [C.POINTER(vp), i32, vp]
        L.ibert_destroy.argtypes = [vp]
        L.ibert_last_status.argtypes = [vp]
        L.ibert_dyadic_from_double.argtypes = [dbl, C.POINTER(C.c_int32), C.POINTER(C.c_int32)]
        L.ibert_linear_i8.argtypes = [vp, vp, dbl, vp, vp, vp, i64, i32, i32, i32, dbl, vp, vp]
        L.ibert_linear_gelu_i8.argtypes = [vp, vp, dbl, vp, vp, vp, i64, i32, i32, dbl, dbl, vp, vp]
        L.ibert_linear_layernorm_i8.argtypes = [vp, vp, dbl, vp, vp, vp, i64, i32, i32, dbl, vp, dbl, vp, vp, dbl,
                                                vp, vp]
        L.ibert_hgelu_i.argtypes = [vp, vp, dbl, i64, dbl, vp, vp]
        L.ibert_gelu_lut_i.argtypes = [vp, vp, dbl, i64, dbl, vp, vp]
        L.ibert_linear_hgelu_i8.argtypes = [vp, vp, dbl, vp, vp, vp, i64, i32, i32, dbl, dbl, vp, vp]
        L.ibert_set_fusion.argtypes = [vp, i32]
        L.ibert_set_split_k.argtypes = [vp, i32]
        L.ibert_set_gelu_table.argtypes = [vp, i32]
        L.ibert_set_gelu_table.restype = i32
        L.ibert_set_qkv_layout.argtypes = [vp, i32]
        L.ibert_set_qkv_layout.restype = i32
        L.ibert_softmax_i.argtypes = [vp, vp, dbl, i64, i32, i32, vp, vp]
        L.ibert_softmax_lut_i.argtypes = [vp, vp, dbl, i64, i32, i32, vp, vp]
        L.ibert_gelu_i.argtypes = [vp, vp, dbl, i64, dbl, vp, vp]
        L.ibert_layernorm_i.argtypes = [vp, vp, dbl, vp, dbl, vp, vp, i64, i32, dbl, vp, vp]
        L.ibert_layernorm_i16.argtypes = [vp, vp, dbl, vp, dbl, vp, vp, i64, i32, dbl, vp, vp]
        L.ibert_layernorm_i16.restype = i32
        L.ibert_attention_i8.argtypes = [vp, vp, i32, i32, i32, i32, dbl, dbl, dbl, dbl, i32, vp, vp]
        L.ibert_attention_masked_i8.argtypes = [vp, vp, i32, i32, i32, i32, vp, dbl, dbl, dbl, dbl, i32, vp, vp]
        L.ibert_encoder_layer_masked.argtypes = [vp, vp, vp, i32, i32, vp, vp, vp]
        L.ibert_embedding_i8.argtypes = [vp, vp, i64, i32, vp, i64, dbl, vp, i64, dbl, vp, vp, i32, dbl, vp, vp]
        L.ibert_classifier_i8.argtypes = [vp, vp, i32, i32, i32, dbl, vp, vp, vp, i32, vp, vp]
        L.ibert_attention_packed_i8.argtypes = [vp, vp, vp, i32, i32, i64, i32, i32, dbl, dbl, dbl, dbl, i32, vp, vp]
        L.ibert_encoder_layer_packed.argtypes = [vp, vp, vp, vp, i32, i32, i64, vp, vp]
        L.ibert_embedding_packed_i8.argtypes = [vp, vp, vp, i32, i32, i64, vp, i64, dbl, vp, i64, dbl, vp, vp, i32, dbl, vp, vp]
        L.ibert_classifier_packed_i8.argtypes = [vp, vp, vp, i32, i32, dbl, vp, vp, vp, i32, vp, vp]
        for name in ("ibert_attention_packed_i8", "ibert_encoder_layer_packed", "ibert_embedding_packed_i8",
                     "ibert_classifier_packed_i8"):
            getattr(L, name).restype = i32
        L.ibert_encoder_graph_create.argtypes = [vp, vp, i32, vp, i32, i32, vp, vp, C.POINTER(vp)]
        L.ibert_encoder_graph_launch.argtypes = [vp, vp]
        L.ibert_encoder_graph_destroy.argtypes = [vp]
        L.ibert_layer_create.argtypes = [vp, C.POINTER(LayerDesc), C.POINTER(vp)]
        L.ibert_layer_destroy.argtypes = [vp]
        L.ibert_encoder_layer.argtypes = [vp, vp, vp, i32, i32, vp, vp]
        L.ibert_layernorm_i_static.argtypes = [vp, vp, dbl, vp, dbl, vp, vp, i64, i32, dbl, vp, vp]
        L.ibert_layernorm_i_static.restype = i32
        L.ibert_layernorm_i_static_status.argtypes = [vp]
        L.ibert_layernorm_i_static_status.restype = i32
        L.ibert_selftest_wait_timeout.argtypes = [vp, i64]
        L.ibert_selftest_wait_timeout.restype = i32
        L.ibert_selftest_exp_division.argtypes = [dbl, C.POINTER(C.c_int32)]
        L.ibert_selftest_exp_division.restype = i32
        L.ibert_profile_begin.argtypes = [vp]
        L.ibert_profile_end.argtypes = [vp, vp, vp]
        L.ibert_profile_begin.restype = i32
        L.ibert_profile_end.restype = i32
        for name in ("ibert_create", "ibert_destroy", "ibert_last_status", "ibert_dyadic_from_double",
                     "ibert_linear_i8", "ibert_linear_gelu_i8", "ibert_linear_layernorm_i8", "ibert_softmax_i", "ibert_gelu_i",
                     "ibert_layernorm_i", "ibert_attention_i8", "ibert_layer_create", "ibert_layer_destroy",
                     "ibert_encoder_layer", "ibert_attention_masked_i8", "ibert_encoder_layer_masked",
                     "ibert_embedding_i8", "ibert_classifier_i8", "ibert_encoder_graph_create",
                     "ibert_encoder_graph_launch", "ibert_encoder_graph_destroy", "ibert_hgelu_i",
                     "ibert_linear_hgelu_i8", "ibert_set_fusion", "ibert_gelu_lut_i", "ibert_softmax_lut_i", "ibert_set_split_k"):
            getattr(L, name).restype = i32
        _lib = L
    return _lib


def _chk(rc: int, where: str):
    if rc != IBERT_OK:
        raise IbertError(rc, where)


def _dev(t: torch.Tensor | None, dtype) -> int | None:
    if t is None:
        return None
    assert t.is_cuda and t.is_contiguous() and t.dtype == dtype, (t.device, t.dtype, dtype)
    return t.data_ptr()


def _host(a, dtype) -> np.ndarray:
    return np.ascontiguousarray(a, dtype=dtype)


def ibert_dyadic_from_double(m: float) -> tuple[int, int]:
    b, c = C.c_int32(), C.c_int32()
    _chk(lib().ibert_dyadic_from_double(m, C.byref(b), C.byref(c)), "ibert_dyadic_from_double")
    return b.value, c.value


def ibert_layernorm_i_static(q: torch.Tensor, S: float, r: torch.Tensor | None, S_r: float, gamma, beta,
                             S_out: float, out: torch.Tensor | None = None, stream: torch.cuda.Stream | None = None):
    """Residual + i-LayerNorm through the entry point that allocates nothing inside the library
    (no context needed; runs on `stream` of the current device)."""
    Cn = q.shape[-1]
    rows = q.numel() // Cn if Cn else 0
    g, b = _host(gamma, np.float64), _host(beta, np.float64)
    if out is None:
        out = torch.empty(q.shape, dtype=torch.int8, device=q.device)
    S_ret = C.c_double()
    sp = None if stream is None else stream.cuda_stream
    _chk(lib().ibert_layernorm_i_static(sp, _dev(q, torch.int32), S, _dev(r, torch.int8), S_r or 0.0,
                                        g.ctypes.data, b.ctypes.data, rows, Cn, S_out, _dev(out, torch.int8),
                                        C.byref(S_ret)), "ibert_layernorm_i_static")
    return out, S_ret.value


def ibert_layernorm_i_static_status(stream: torch.cuda.Stream | None = None) -> int:
    """Synchronizes `stream` and returns (then clears) the device-side status of the
    allocation-free LayerNorm calls on the current device."""
    return int(lib().ibert_layernorm_i_static_status(None if stream is None else stream.cuda_stream))


class Context:
    """``ibert_ctx``: a device and the stream every call is enqueued on."""

    def __init__(self, device: int = 0, stream: torch.cuda.Stream | None = None):
        self.device = device
        self.stream = stream
        h = C.c_void_p()
        sp = None if stream is None else stream.cuda_stream
        _chk(lib().ibert_create(C.byref(h), device, sp), "ibert_create")
        self.h = h

    def close(self):
        if self.h:
            lib().ibert_destroy(self.h)
            self.h = None

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass

    def ibert_last_status(self) -> int:
        return int(lib().ibert_last_status(self.h))

    def ibert_set_fusion(self, mode: int):
        """0: linear + LayerNorm fusion by problem size (default), 1: whenever supported, 2: never."""
        _chk(lib().ibert_set_fusion(self.h, mode), "ibert_set_fusion")

    def ibert_set_split_k(self, mode: int) -> None:
        """0: split K of small GEMMs by size (default); 1: never; 2 / 4: force that cluster width."""
        _chk(lib().ibert_set_split_k(self.h, mode), "ibert_set_split_k")

    def ibert_set_qkv_layout(self, mode: int) -> None:
        """0: the layer keeps Q | K | V and the FFN1 result transposed between its kernels where shapes allow and sizes make it pay (default); 1: never; 2: wherever shapes allow."""
        _chk(lib().ibert_set_qkv_layout(self.h, mode), "ibert_set_qkv_layout")

    def ibert_set_gelu_table(self, mode: int) -> None:
        """0: FFN1's i-GELU from the layer's table where the tile shape has room (default); 1: computed."""
        _chk(lib().ibert_set_gelu_table(self.h, mode), "ibert_set_gelu_table")

    def check(self):
        _chk(self.ibert_last_status(), "ibert_last_status")

    def ibert_selftest_wait_timeout(self, limit_us: int) -> None:
        """Enqueues the one-warp kernel whose bounded wait runs out after `limit_us` microseconds."""
        _chk(lib().ibert_selftest_wait_timeout(self.h, limit_us), "ibert_selftest_wait_timeout")

    def ibert_profile_begin(self):
        _chk(lib().ibert_profile_begin(self.h), "ibert_profile_begin")

    def ibert_profile_end(self) -> dict:
        """{kernel class name: (device ms summed, launches)} for the launches since profile_begin."""
        ms = np.zeros(len(KERNEL_CLASSES), dtype=np.float32)
        n = np.zeros(len(KERNEL_CLASSES), dtype=np.int32)
        _chk(lib().ibert_profile_end(self.h, ms.ctypes.data, n.ctypes.data), "ibert_profile_end")
        return {k: (float(ms[i]), int(n[i])) for i, k in enumerate(KERNEL_CLASSES)}

    # ------------------------------------------------------------------ simple ops
    def ibert_gelu_i(self, q: torch.Tensor, S: float, S_out: float, out: torch.Tensor | None = None):
        if out is None:
            out = torch.empty(q.shape, dtype=torch.int8, device=q.device)
        S_ret = C.c_double()
        _chk(lib().ibert_gelu_i(self.h, _dev(q, torch.int32), S, q.numel(), S_out, _dev(out, torch.int8),
                                C.byref(S_ret)), "ibert_gelu_i")
        return out, S_ret.value

    def ibert_gelu_lut_i(self, q: torch.Tensor, S: float, S_out: float, out: torch.Tensor | None = None):
        """i-GELU through a look-up table built from the integer kernel (comparison only)."""
        if out is None:
            out = torch.empty(q.shape, dtype=torch.int8, device=q.device)
        S_ret = C.c_double()
        _chk(lib().ibert_gelu_lut_i(self.h, _dev(q, torch.int32), S, q.numel(), S_out, _dev(out, torch.int8),
                                    C.byref(S_ret)), "ibert_gelu_lut_i")
        return out, S_ret.value

    def ibert_hgelu_i(self, q: torch.Tensor, S: float, S_out: float, out: torch.Tensor | None = None):
        """Integer h-GELU (Eq. 6), the paper's comparison function."""
        if out is None:
            out = torch.empty(q.shape, dtype=torch.int8, device=q.device)
        S_ret = C.c_double()
        _chk(lib().ibert_hgelu_i(self.h, _dev(q, torch.int32), S, q.numel(), S_out, _dev(out, torch.int8),
                                 C.byref(S_ret)), "ibert_hgelu_i")
        return out, S_ret.value

    def ibert_softmax_i(self, q: torch.Tensor, S: float, p_max: int = 255, out: torch.Tensor | None = None,
                        _entry: str = "ibert_softmax_i"):
        L = q.shape[-1]
        rows = q.numel() // L if L else 0
        if out is None:
            out = torch.empty(q.shape, dtype=torch.uint8, device=q.device)
        S_ret = C.c_double()
        _chk(getattr(lib(), _entry)(self.h, _dev(q, torch.int32), S, rows, L, p_max, _dev(out, torch.uint8),
                                    C.byref(S_ret)), _entry)
        return out, S_ret.value

    def ibert_softmax_lut_i(self, q: torch.Tensor, S: float, p_max: int = 255, out: torch.Tensor | None = None):
        """i-softmax with i-exp read from a table built by the integer function (comparison only)."""
        return self.ibert_softmax_i(q, S, p_max, out, _entry="ibert_softmax_lut_i")

    def ibert_layernorm_i(self, q: torch.Tensor, S: float, r: torch.Tensor | None, S_r: float, gamma, beta,
                          S_out: float, out: torch.Tensor | None = None):
        Cn = q.shape[-1]
        rows = q.numel() // Cn if Cn else 0
        g, b = _host(gamma, np.float64), _host(beta, np.float64)
        assert g.size == Cn and b.size == Cn
        if out is None:
            out = torch.empty(q.shape, dtype=torch.int8, device=q.device)
        S_ret = C.c_double()
        if q.dtype == torch.int16:           # Q16 values in an int16 container
            _chk(lib().ibert_layernorm_i16(self.h, _dev(q, torch.int16), S, _dev(r, torch.int8), S_r or 0.0,
                                           g.ctypes.data, b.ctypes.data, rows, Cn, S_out, _dev(out, torch.int8),
                                           C.byref(S_ret)), "ibert_layernorm_i16")
            return out, S_ret.value
        _chk(lib().ibert_layernorm_i(self.h, _dev(q, torch.int32), S, _dev(r, torch.int8), S_r or 0.0,
                                     g.ctypes.data, b.ctypes.data, rows, Cn, S_out, _dev(out, torch.int8),
                                     C.byref(S_ret)), "ibert_layernorm_i")
        return out, S_ret.value

    def ibert_linear_i8(self, x: torch.Tensor, S_x: float, w: torch.Tensor, S_w, bias: torch.Tensor | None,
                        out_kind: int, S_out: float = 1.0, out: torch.Tensor | None = None):
        K = x.shape[-1]
        M = x.numel() // K
        N = w.shape[0]
        assert w.shape[1] == K
        sw = _host(S_w, np.float64)
        assert sw.size == N
        if out is None:
            out = torch.empty(x.shape[:-1] + (N,), device=x.device,
                              dtype={0: torch.int8, 3: torch.int16}.get(out_kind, torch.int32))
        S_ret = np.zeros(N if out_kind == 2 else 1, dtype=np.float64)
        _chk(lib().ibert_linear_i8(self.h, _dev(x, torch.int8), S_x, _dev(w, torch.int8), sw.ctypes.data,
                                   _dev(bias, torch.int32), M, N, K, out_kind, S_out, out.data_ptr(),
                                   S_ret.ctypes.data), "ibert_linear_i8")
        return out, (S_ret if out_kind == 2 else float(S_ret[0]))

    def ibert_linear_hgelu_i8(self, x: torch.Tensor, S_x: float, w: torch.Tensor, S_w, bias: torch.Tensor | None,
                              S_mid: float, S_out: float, out: torch.Tensor | None = None):
        K = x.shape[-1]
        M = x.numel() // K
        N = w.shape[0]
        sw = _host(S_w, np.float64)
        if out is None:
            out = torch.empty(x.shape[:-1] + (N,), dtype=torch.int8, device=x.device)
        S_ret = C.c_double()
        _chk(lib().ibert_linear_hgelu_i8(self.h, _dev(x, torch.int8), S_x, _dev(w, torch.int8), sw.ctypes.data,
                                         _dev(bias, torch.int32), M, N, K, S_mid, S_out, _dev(out, torch.int8),
                                         C.byref(S_ret)), "ibert_linear_hgelu_i8")
        return out, S_ret.value

    def ibert_linear_layernorm_i8(self, x: torch.Tensor, S_x: float, w: torch.Tensor, S_w,
                                  bias: torch.Tensor | None, S_mid: float, res: torch.Tensor, S_res: float,
                                  gamma, beta, S_out: float, out: torch.Tensor | None = None):
        """Linear layer (Q16 at S_mid) + residual + i-LayerNorm as one call."""
        K = x.shape[-1]
        M = x.numel() // K
        N = w.shape[0]
        assert w.shape[1] == K and res.numel() == M * N
        sw = _host(S_w, np.float64)
        g, b = _host(gamma, np.float64), _host(beta, np.float64)
        assert sw.size == N and g.size == N and b.size == N
        if out is None:
            out = torch.empty(x.shape[:-1] + (N,), dtype=torch.int8, device=x.device)
        S_ret = C.c_double()
        _chk(lib().ibert_linear_layernorm_i8(self.h, _dev(x, torch.int8), S_x, _dev(w, torch.int8), sw.ctypes.data,
                                             _dev(bias, torch.int32), M, N, K, S_mid, _dev(res, torch.int8), S_res,
                                             g.ctypes.data, b.ctypes.data, S_out, _dev(out, torch.int8),
                                             C.byref(S_ret)), "ibert_linear_layernorm_i8")
        return out, S_ret.value

    def ibert_linear_gelu_i8(self, x: torch.Tensor, S_x: float, w: torch.Tensor, S_w, bias: torch.Tensor | None,
                             S_mid: float, S_out: float, out: torch.Tensor | None = None):
        K = x.shape[-1]
        M = x.numel() // K
        N = w.shape[0]
        sw = _host(S_w, np.float64)
        if out is None:
            out = torch.empty(x.shape[:-1] + (N,), dtype=torch.int8, device=x.device)
        S_ret = C.c_double()
        _chk(lib().ibert_linear_gelu_i8(self.h, _dev(x, torch.int8), S_x, _dev(w, torch.int8), sw.ctypes.data,
                                        _dev(bias, torch.int32), M, N, K, S_mid, S_out, _dev(out, torch.int8),
                                        C.byref(S_ret)), "ibert_linear_gelu_i8")
        return out, S_ret.value

    def ibert_attention_i8(self, qkv: torch.Tensor, B: int, L: int, H: int, heads: int, S_q: float, S_k: float,
                           S_v: float, S_ctx: float, p_max: int = 255, out: torch.Tensor | None = None):
        assert qkv.numel() == B * L * 3 * H
        if out is None:
            out = torch.empty((B * L, H), dtype=torch.int8, device=qkv.device)
        S_ret = C.c_double()
        _chk(lib().ibert_attention_i8(self.h, _dev(qkv, torch.int8), B, L, H, heads, S_q, S_k, S_v, S_ctx, p_max,
                                      _dev(out, torch.int8), C.byref(S_ret)), "ibert_attention_i8")
        return out, S_ret.value

    def ibert_attention_masked_i8(self, qkv: torch.Tensor, B: int, L: int, H: int, heads: int, lens: torch.Tensor,
                                  S_q: float, S_k: float, S_v: float, S_ctx: float, p_max: int = 255,
                                  out: torch.Tensor | None = None):
        """Attention with a key-padding mask; ``lens``: device int32 [B], valid keys per sequence."""
        assert qkv.numel() == B * L * 3 * H and lens.numel() == B
        if out is None:
            out = torch.empty((B * L, H), dtype=torch.int8, device=qkv.device)
        S_ret = C.c_double()
        _chk(lib().ibert_attention_masked_i8(self.h, _dev(qkv, torch.int8), B, L, H, heads, _dev(lens, torch.int32),
                                             S_q, S_k, S_v, S_ctx, p_max, _dev(out, torch.int8), C.byref(S_ret)),
             "ibert_attention_masked_i8")
        return out, S_ret.value

    def ibert_embedding_i8(self, ids: torch.Tensor, L: int, word: torch.Tensor, S_word: float, pos: torch.Tensor,
                           S_pos: float, gamma, beta, S_out: float, out: torch.Tensor | None = None):
        """INT8 word + position embedding followed by i-LayerNorm (token t: position t mod L)."""
        T = ids.numel()
        V, H = word.shape
        P = pos.shape[0]
        g, b = _host(gamma, np.float64), _host(beta, np.float64)
        assert pos.shape[1] == H and g.size == H and b.size == H
        if out is None:
            out = torch.empty((T, H), dtype=torch.int8, device=word.device)
        S_ret = C.c_double()
        _chk(lib().ibert_embedding_i8(self.h, _dev(ids, torch.int32), T, L, _dev(word, torch.int8), V, S_word,
                                      _dev(pos, torch.int8), P, S_pos, g.ctypes.data, b.ctypes.data, H, S_out,
                                      _dev(out, torch.int8), C.byref(S_ret)), "ibert_embedding_i8")
        return out, S_ret.value

    def ibert_classifier_i8(self, x: torch.Tensor, B: int, L: int, S_x: float, w: torch.Tensor, S_w,
                            bias: torch.Tensor | None, out: torch.Tensor | None = None):
        """Raw INT32 logits of a linear head on the first token of every sequence."""
        N, H = w.shape
        assert x.numel() == B * L * H
        sw = _host(S_w, np.float64)
        assert sw.size == N
        if out is None:
            out = torch.empty((B, N), dtype=torch.int32, device=x.device)
        S_ret = np.zeros(N, dtype=np.float64)
        _chk(lib().ibert_classifier_i8(self.h, _dev(x, torch.int8), B, L, H, S_x, _dev(w, torch.int8), sw.ctypes.data,
                                       _dev(bias, torch.int32), N, _dev(out, torch.int32), S_ret.ctypes.data),
             "ibert_classifier_i8")
        return out, S_ret

    # ------------------------------------------------------------------ packed batches
    def ibert_attention_packed_i8(self, qkv: torch.Tensor, cu_seqlens: torch.Tensor, max_len: int, H: int, heads: int,
                                  S_q: float, S_k: float, S_v: float, S_ctx: float, p_max: int = 255,
                                  out: torch.Tensor | None = None):
        """Attention on a packed batch; ``cu_seqlens``: device int32 [B + 1], first rows of the sequences."""
        B = cu_seqlens.numel() - 1
        total = qkv.numel() // (3 * H)
        if out is None:
            out = torch.empty((total, H), dtype=torch.int8, device=qkv.device)
        S_ret = C.c_double()
        _chk(lib().ibert_attention_packed_i8(self.h, _dev(qkv, torch.int8), _dev(cu_seqlens, torch.int32), B, max_len,
                                             total, H, heads, S_q, S_k, S_v, S_ctx, p_max, _dev(out, torch.int8),
                                             C.byref(S_ret)), "ibert_attention_packed_i8")
        return out, S_ret.value

    def ibert_encoder_layer_packed(self, layer: "Layer", x: torch.Tensor, cu_seqlens: torch.Tensor, max_len: int,
                                   out: torch.Tensor | None = None):
        """The encoder layer on a packed batch [total tokens, H]."""
        B = cu_seqlens.numel() - 1
        total = x.numel() // layer.H
        if out is None:
            out = torch.empty((total, layer.H), dtype=torch.int8, device=x.device)
        S_ret = C.c_double()
        _chk(lib().ibert_encoder_layer_packed(self.h, layer.h, _dev(x, torch.int8), _dev(cu_seqlens, torch.int32), B,
                                              max_len, total, _dev(out, torch.int8), C.byref(S_ret)),
             "ibert_encoder_layer_packed")
        return out, S_ret.value

    def ibert_embedding_packed_i8(self, ids: torch.Tensor, cu_seqlens: torch.Tensor, max_len: int, word: torch.Tensor,
                                  S_word: float, pos: torch.Tensor, S_pos: float, gamma, beta, S_out: float,
                                  out: torch.Tensor | None = None):
        T = ids.numel()
        B = cu_seqlens.numel() - 1
        V, H = word.shape
        g, b = _host(gamma, np.float64), _host(beta, np.float64)
        if out is None:
            out = torch.empty((T, H), dtype=torch.int8, device=word.device)
        S_ret = C.c_double()
        _chk(lib().ibert_embedding_packed_i8(self.h, _dev(ids, torch.int32), _dev(cu_seqlens, torch.int32), B, max_len, T,
                                             _dev(word, torch.int8), V, S_word, _dev(pos, torch.int8), pos.shape[0],
                                             S_pos, g.ctypes.data, b.ctypes.data, H, S_out, _dev(out, torch.int8),
                                             C.byref(S_ret)), "ibert_embedding_packed_i8")
        return out, S_ret.value

    def ibert_classifier_packed_i8(self, x: torch.Tensor, cu_seqlens: torch.Tensor, S_x: float, w: torch.Tensor, S_w,
                                   bias: torch.Tensor | None, out: torch.Tensor | None = None):
        N, H = w.shape
        B = cu_seqlens.numel() - 1
        sw = _host(S_w, np.float64)
        if out is None:
            out = torch.empty((B, N), dtype=torch.int32, device=x.device)
        S_ret = np.zeros(N, dtype=np.float64)
        _chk(lib().ibert_classifier_packed_i8(self.h, _dev(x, torch.int8), _dev(cu_seqlens, torch.int32), B, H, S_x,
                                              _dev(w, torch.int8), sw.ctypes.data, _dev(bias, torch.int32), N,
                                              _dev(out, torch.int32), S_ret.ctypes.data), "ibert_classifier_packed_i8")
        return out, S_ret

    # ------------------------------------------------------------------ encoder layer
    def ibert_layer_create(self, params: dict) -> "Layer":
        return Layer(self, params)

    def ibert_encoder_layer(self, layer: "Layer", x: torch.Tensor, B: int, L: int,
                            out: torch.Tensor | None = None):
        if out is None:
            out = torch.empty((B * L, layer.H), dtype=torch.int8, device=x.device)
        S_ret = C.c_double()
        _chk(lib().ibert_encoder_layer(self.h, layer.h, _dev(x, torch.int8), B, L, _dev(out, torch.int8),
                                       C.byref(S_ret)), "ibert_encoder_layer")
        return out, S_ret.value

    def ibert_encoder_layer_masked(self, layer: "Layer", x: torch.Tensor, B: int, L: int, lens: torch.Tensor,
                                   out: torch.Tensor | None = None):
        """The encoder layer on padded sequences; ``lens``: device int32 [B], valid keys per sequence."""
        assert lens.numel() == B
        if out is None:
            out = torch.empty((B * L, layer.H), dtype=torch.int8, device=x.device)
        S_ret = C.c_double()
        _chk(lib().ibert_encoder_layer_masked(self.h, layer.h, _dev(x, torch.int8), B, L, _dev(lens, torch.int32),
                                              _dev(out, torch.int8), C.byref(S_ret)), "ibert_encoder_layer_masked")
        return out, S_ret.value


class Graph:
    """``ibert_graph``: a stack of encoder layers captured into a CUDA graph for fixed shapes and
    fixed buffers (``x`` in, ``out`` out, optional ``lens``); ``launch()`` replays it."""

    def __init__(self, ctx: "Context", layers, x: torch.Tensor, B: int, L: int, out: torch.Tensor,
                 lens: torch.Tensor | None = None):
        self.ctx = ctx
        self.keep = (list(layers), x, out, lens)          # the graph refers to these buffers
        arr = (C.c_void_p * len(layers))(*[ly.h for ly in layers])
        h = C.c_void_p()
        _chk(lib().ibert_encoder_graph_create(ctx.h, arr, len(layers), _dev(x, torch.int8), B, L,
                                              _dev(lens, torch.int32), _dev(out, torch.int8), C.byref(h)),
             "ibert_encoder_graph_create")
        self.h = h
        self.out = out

    def launch(self) -> torch.Tensor:
        _chk(lib().ibert_encoder_graph_launch(self.ctx.h, self.h), "ibert_encoder_graph_launch")
        return self.out

    def close(self):
        if self.h:
            lib().ibert_encoder_graph_destroy(self.h)
            self.h = None


class Layer:
    """``ibert_layer``: device-resident integer parameters of one encoder layer, built from the
    dictionary of host arrays a synthetic-layer generator (or a calibrated checkpoint) provides."""

    def __init__(self, ctx: Context, params: dict):
        self.ctx = ctx
        self.H = int(params["H"])
        d = LayerDesc()
        d.H, d.heads, d.F, d.p_max = self.H, int(params["heads"]), int(params["F"]), int(params["p_max"])
        keep = []

        def ptr(name, dtype):
            a = _host(params[name], dtype)
            keep.append(a)
            return a.ctypes.data

        for nm in ("qkv", "o", "f1", "f2"):
            setattr(d, f"w_{nm}", ptr(f"w_{nm}", np.int8))
            setattr(d, f"S_w_{nm}", ptr(f"S_w_{nm}", np.float64))
            setattr(d, f"bias_{nm}", ptr(f"bias_{nm}", np.int32))
        for nm in ("gamma1", "beta1", "gamma2", "beta2"):
            setattr(d, nm, ptr(nm, np.float64))
        for nm in SCALE_NAMES:
            setattr(d, nm, float(params[nm]))
        h = C.c_void_p()
        _chk(lib().ibert_layer_create(ctx.h, C.byref(d), C.byref(h)), "ibert_layer_create")
        self.h = h

    def close(self):
        if self.h and self.ctx.h:
            lib().ibert_layer_destroy(self.h)
        self.h = None

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass
