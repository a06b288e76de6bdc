"""ctypes front end of the CPU oracle (``ibert_oracle.c``).

TEST INFRASTRUCTURE ONLY: nothing on the product path may import this
package.  It compiles the C file with gcc on first use (``build()``) and
exposes each oracle function on numpy arrays.  No arithmetic of the method
lives here -- only argument marshalling.
"""
from __future__ import annotations

import ctypes as C
import os
import subprocess
from dataclasses import dataclass
from pathlib import Path

import numpy as np

_HERE = Path(__file__).resolve().parent
_SRC = _HERE / "ibert_oracle.c"
_LIB = _HERE / "libibert_oracle.so"
_lib = None


class OracleError(RuntimeError):
    def __init__(self, code: int, where: str):
        super().__init__(f"oracle {where} failed with code {code}")
        self.code = code


def build(force: bool = False) -> Path:
    """Compile the oracle (gcc -O2, OpenMP, no FMA contraction)."""
    import hashlib
    digest = hashlib.sha256(_SRC.read_bytes()).hexdigest()
    stamp = _LIB.with_suffix(".so.srchash")
    # (file times do not survive a copy of the tree: compare a hash of the source instead)
    if force or not _LIB.exists() or not stamp.exists() or stamp.read_text().strip() != digest:
        tmp = _LIB.with_suffix(f".tmp{os.getpid()}.so")
        subprocess.check_call(
            ["gcc", "-O2", "-std=c11", "-fopenmp", "-ffp-contract=off", "-fno-fast-math",
             "-fPIC", "-shared", "-Wall", "-Wno-maybe-uninitialized", "-o", str(tmp), str(_SRC), "-lm"])
        os.replace(tmp, _LIB)
        stamp.write_text(digest + "\n")
    return _LIB


def lib():
    global _lib
    if _lib is None:
        build()
        _lib = C.CDLL(str(_LIB))
        _lib.orc_requant.restype = C.c_int64
        _lib.orc_requant.argtypes = [C.c_int64, C.c_int64, C.c_int, C.c_int64]
        _lib.orc_round_shift.restype = C.c_int64
        _lib.orc_round_shift.argtypes = [C.c_int64, C.c_int]
        _lib.orc_isqrt.restype = C.c_int64
        _lib.orc_isqrt.argtypes = [C.c_int64, C.POINTER(C.c_int)]
    return _lib


def _chk(rc: int, where: str):
    if rc != 0:
        raise OracleError(rc, where)


def _p(a: np.ndarray | None):
    return None if a is None else a.ctypes.data_as(C.c_void_p)


def _arr(a, dtype):
    return np.ascontiguousarray(a, dtype=dtype)


def num_threads() -> int:
    return int(lib().orc_num_threads())


# ------------------------------------------------------------------ requant
def dyadic(m: float) -> tuple[int, int]:
    b = C.c_int64()
    c = C.c_int()
    _chk(lib().orc_dyadic(C.c_double(m), C.byref(b), C.byref(c)), "dyadic")
    return int(b.value), int(c.value)


def round_shift(v: int, c: int) -> int:
    return int(lib().orc_round_shift(v, c))


def requant(v: int, b: int, c: int, qmax: int) -> int:
    return int(lib().orc_requant(v, b, c, qmax))


# ------------------------------------------------------------------ isqrt
def isqrt(n: int) -> tuple[int, int]:
    """Returns (floor(sqrt(n)), number of integer divisions Algorithm 4 used)."""
    d = C.c_int()
    r = lib().orc_isqrt(n, C.byref(d))
    return int(r), int(d.value)


# ------------------------------------------------------------------ i-exp / softmax
class _ExpConsts(C.Structure):
    _fields_ = [("s_in", C.c_int), ("q_ln2", C.c_int64), ("q_b", C.c_int64), ("q_c", C.c_int64),
                ("e_top", C.c_int64), ("s_out", C.c_int), ("S_e", C.c_double)]


def exp_consts(S: float) -> dict:
    k = _ExpConsts()
    _chk(lib().orc_exp_consts_from_scale(C.c_double(S), C.byref(k)), "exp_consts")
    return {f: getattr(k, f) for f, _ in _ExpConsts._fields_}


def iexp(q_tilde, S: float) -> tuple[np.ndarray, float]:
    q = _arr(q_tilde, np.int64)
    e = np.empty_like(q)
    S_e = C.c_double()
    _chk(lib().orc_iexp(_p(q), C.c_int64(q.size), C.c_double(S), _p(e), C.byref(S_e)), "iexp")
    return e, float(S_e.value)


def softmax(q, S: float, p_max: int = 255) -> tuple[np.ndarray, float]:
    q = _arr(q, np.int32)
    L = q.shape[-1]
    rows = q.size // L if L else 0
    out = np.empty(q.shape, dtype=np.uint8)
    S_ret = C.c_double()
    _chk(lib().orc_softmax(_p(q), C.c_double(S), C.c_int64(rows), C.c_int(L), C.c_int(p_max),
                           _p(out), C.byref(S_ret)), "softmax")
    return out, float(S_ret.value)


# ------------------------------------------------------------------ i-GELU
class _GeluConsts(C.Structure):
    _fields_ = [("s_in", C.c_int), ("q_b", C.c_int64), ("q_c", C.c_int64), ("S_erf", C.c_double),
                ("s_f", C.c_int), ("S_g", C.c_double)]


def gelu_consts(S: float) -> dict:
    k = _GeluConsts()
    _chk(lib().orc_gelu_consts_from_scale(C.c_double(S), C.byref(k)), "gelu_consts")
    return {f: getattr(k, f) for f, _ in _GeluConsts._fields_}


def gelu_raw(q, S: float) -> tuple[np.ndarray, float]:
    q = _arr(q, np.int32)
    g = np.empty(q.shape, dtype=np.int64)
    S_g = C.c_double()
    _chk(lib().orc_gelu_raw(_p(q), C.c_double(S), C.c_int64(q.size), _p(g), C.byref(S_g)), "gelu_raw")
    return g, float(S_g.value)


def gelu(q, S: float, S_out: float) -> tuple[np.ndarray, float]:
    q = _arr(q, np.int32)
    out = np.empty(q.shape, dtype=np.int8)
    S_ret = C.c_double()
    _chk(lib().orc_gelu(_p(q), C.c_double(S), C.c_int64(q.size), C.c_double(S_out), _p(out),
                        C.byref(S_ret)), "gelu")
    return out, float(S_ret.value)


def hgelu(q, S: float, S_out: float) -> tuple[np.ndarray, float]:
    """Integer h-GELU (Eq. 6: x ReLU6(1.702 x + 3) / 6), the comparison function of Table 1."""
    q = _arr(q, np.int32)
    out = np.empty(q.shape, dtype=np.int8)
    S_ret = C.c_double()
    _chk(lib().orc_hgelu(_p(q), C.c_double(S), C.c_int64(q.size), C.c_double(S_out), _p(out),
                         C.byref(S_ret)), "hgelu")
    return out, float(S_ret.value)


# ------------------------------------------------------------------ i-LayerNorm
def layernorm(q, S: float, r, S_r: float, gamma, beta, S_out: float) -> tuple[np.ndarray, float]:
    q = _arr(q, np.int32)
    Cn = q.shape[-1]
    rows = q.size // Cn
    r = None if r is None else _arr(r, np.int8)
    gamma = _arr(gamma, np.float64)
    beta = _arr(beta, np.float64)
    assert gamma.size == Cn and beta.size == Cn
    out = np.empty(q.shape, dtype=np.int8)
    S_ret = C.c_double()
    _chk(lib().orc_layernorm(_p(q), C.c_double(S), _p(r), C.c_double(S_r), _p(gamma), _p(beta),
                             C.c_int64(rows), C.c_int(Cn), C.c_double(S_out), _p(out),
                             C.byref(S_ret)), "layernorm")
    return out, float(S_ret.value)


# ------------------------------------------------------------------ linear
def linear(x, S_x: float, w, S_w, bias, out_kind: int, S_out: float = 0.0, S_out_cols=None):
    x = _arr(x, np.int8)
    w = _arr(w, np.int8)
    K = x.shape[-1]
    M = x.size // K
    N = w.shape[0]
    assert w.shape[1] == K
    S_w = _arr(S_w, np.float64)
    bias = None if bias is None else _arr(bias, np.int32)
    S_out_cols = None if S_out_cols is None else _arr(S_out_cols, np.float64)
    out = np.empty(x.shape[:-1] + (N,), dtype=np.int8 if out_kind == 0 else np.int32)
    _chk(lib().orc_linear(_p(x), C.c_double(S_x), _p(w), _p(S_w), _p(bias), C.c_int64(M), C.c_int(N),
                          C.c_int(K), C.c_int(out_kind), C.c_double(S_out), _p(S_out_cols), _p(out)),
         "linear")
    return out


# ------------------------------------------------------------------ attention
def attention(qkv, B: int, L: int, H: int, heads: int, S_q: float, S_k: float, S_v: float,
              S_ctx: float, p_max: int = 255, want_probs: bool = False, lens=None):
    """``lens`` (optional, [B] int32): valid keys per sequence (key-padding mask)."""
    qkv = _arr(qkv, np.int8)
    assert qkv.size == B * L * 3 * H
    ctx = np.empty((B * L, H), dtype=np.int8)
    probs = np.empty((B, heads, L, L), dtype=np.uint8) if want_probs else None
    if lens is None:
        _chk(lib().orc_attention(_p(qkv), C.c_int(B), C.c_int(L), C.c_int(H), C.c_int(heads),
                                 C.c_double(S_q), C.c_double(S_k), C.c_double(S_v), C.c_double(S_ctx),
                                 C.c_int(p_max), _p(ctx), _p(probs)), "attention")
    else:
        lens = _arr(lens, np.int32)
        assert lens.size == B
        _chk(lib().orc_attention_masked(_p(qkv), C.c_int(B), C.c_int(L), C.c_int(H), C.c_int(heads), _p(lens),
                                        C.c_double(S_q), C.c_double(S_k), C.c_double(S_v), C.c_double(S_ctx),
                                        C.c_int(p_max), _p(ctx), _p(probs)), "attention_masked")
    return (ctx, probs) if want_probs else ctx


# ------------------------------------------------------------------ encoder layer
class _LayerDesc(C.Structure):
    _fields_ = [("H", C.c_int), ("heads", C.c_int), ("F", C.c_int), ("p_max", C.c_int)] + [
        (n, C.c_void_p) for n in (
            "w_qkv", "S_w_qkv", "bias_qkv", "w_o", "S_w_o", "bias_o",
            "w_f1", "S_w_f1", "bias_f1", "w_f2", "S_w_f2", "bias_f2",
            "gamma1", "beta1", "gamma2", "beta2")] + [
        (n, C.c_double) for n in (
            "S_x", "S_q", "S_k", "S_v", "S_ctx", "S_r1", "S_h1", "S_gi", "S_go", "S_r2", "S_out")]


class _LayerTaps(C.Structure):
    _fields_ = [(n, C.c_void_p) for n in ("qkv", "ctx", "r1", "h1", "g", "r2")]


SCALE_NAMES = ("S_x", "S_q", "S_k", "S_v", "S_ctx", "S_r1", "S_h1", "S_gi", "S_go", "S_r2", "S_out")


@dataclass
class LayerResult:
    out: np.ndarray
    taps: dict


def encoder_layer(params: dict, x, B: int, L: int, want_taps: bool = False, lens=None) -> LayerResult:
    """``params``: the dictionary a synthetic-layer generator produces (int8 weights,
    per-channel weight scales, int32 biases, gamma/beta, the 11 activation scales)."""
    H, F = int(params["H"]), int(params["F"])
    keep = []

    def ptr(name, dtype):
        a = _arr(params[name], dtype)
        keep.append(a)
        return a.ctypes.data

    d = _LayerDesc()
    d.H, d.heads, d.F, d.p_max = H, int(params["heads"]), F, int(params["p_max"])
    for nm in ("qkv", "o", "f1", "f2"):
        setattr(d, f"w_{nm}", ptr(f"w_{nm}", np.int8))
        setattr(d, f"S_w_{nm}", ptr(f"S_w_{nm}", np.float64))
        setattr(d, f"bias_{nm}", ptr(f"bias_{nm}", np.int32))
    for nm in ("gamma1", "beta1", "gamma2", "beta2"):
        setattr(d, nm, ptr(nm, np.float64))
    for nm in SCALE_NAMES:
        setattr(d, nm, float(params[nm]))
    x = _arr(x, np.int8)
    T = B * L
    assert x.size == T * H
    out = np.empty((T, H), dtype=np.int8)
    taps = {}
    tp = None
    if want_taps:
        taps = {"qkv": np.empty((T, 3 * H), np.int8), "ctx": np.empty((T, H), np.int8),
                "r1": np.empty((T, H), np.int32), "h1": np.empty((T, H), np.int8),
                "g": np.empty((T, F), np.int8), "r2": np.empty((T, H), np.int32)}
        t = _LayerTaps()
        for k, v in taps.items():
            setattr(t, k, v.ctypes.data)
        tp = C.byref(t)
    if lens is None:
        _chk(lib().orc_encoder_layer(C.byref(d), _p(x), C.c_int(B), C.c_int(L), _p(out), tp),
             "encoder_layer")
    else:
        lens = _arr(lens, np.int32)
        assert lens.size == B
        _chk(lib().orc_encoder_layer_masked(C.byref(d), _p(x), C.c_int(B), C.c_int(L), _p(lens), _p(out), tp),
             "encoder_layer_masked")
    return LayerResult(out=out, taps=taps)


# ------------------------------------------------------------------ around the layers
def embedding(ids, L: int, word, S_word: float, pos, S_pos: float, gamma, beta, S_out: float) -> np.ndarray:
    """INT8 word + position embedding followed by i-LayerNorm; token t uses position t mod L."""
    ids = _arr(ids, np.int32)
    word = _arr(word, np.int8)
    pos = _arr(pos, np.int8)
    V, H = word.shape
    P = pos.shape[0]
    assert pos.shape[1] == H
    gamma = _arr(gamma, np.float64)
    beta = _arr(beta, np.float64)
    T = ids.size
    out = np.empty((T, H), dtype=np.int8)
    _chk(lib().orc_embedding(_p(ids), C.c_int64(T), C.c_int(L), _p(word), C.c_int64(V), C.c_double(S_word),
                             _p(pos), C.c_int64(P), C.c_double(S_pos), _p(gamma), _p(beta), C.c_int(H),
                             C.c_double(S_out), _p(out)), "embedding")
    return out


def classifier(x, B: int, L: int, S_x: float, w, S_w, bias) -> np.ndarray:
    """Raw INT32 logits of a linear head on the first token of every sequence."""
    x = _arr(x, np.int8)
    w = _arr(w, np.int8)
    N, H = w.shape
    assert x.size == B * L * H
    S_w = _arr(S_w, np.float64)
    bias = None if bias is None else _arr(bias, np.int32)
    logits = np.empty((B, N), dtype=np.int32)
    _chk(lib().orc_classifier(_p(x), C.c_int(B), C.c_int(L), C.c_int(H), C.c_double(S_x), _p(w), _p(S_w),
                              _p(bias), C.c_int(N), _p(logits)), "classifier")
    return logits
