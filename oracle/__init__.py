"""ctypes loader for the float64 CPU oracle (``sprinter_oracle.c``).

TEST INFRASTRUCTURE ONLY: the CUDA library never imports this package, and this
package imports nothing from it.  Arrays are numpy; bfloat16 tensors are passed
as their raw ``uint16`` bit patterns.

Element type is inferred from the numpy dtype: float32 -> 0, uint16 (bf16
bits) -> 1, float64 -> 2.
"""
from __future__ import annotations

import ctypes as C
import os
import subprocess

import numpy as np

_DIR = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_DIR, "sprinter_oracle.c")
_LIB = os.path.join(_DIR, "libsprinter_oracle.so")

OK, ERR_ARG, ERR_TOKEN, ERR_ROW = 0, 1, 6, 7


def build(force: bool = False) -> str:
    """Compile the oracle with gcc (-O2, no fast-math) if the library is stale."""
    if force or not os.path.exists(_LIB) or os.path.getmtime(_LIB) < os.path.getmtime(_SRC):
        tmp = _LIB + f".tmp{os.getpid()}"
        subprocess.check_call(
            ["gcc", "-O2", "-std=c99", "-fPIC", "-shared", "-o", tmp, _SRC, "-lm"])
        os.replace(tmp, _LIB)
    return _LIB


_lib = None


def lib():
    global _lib
    if _lib is None:
        L = C.CDLL(build())
        vp, i32, i64, f32, f64 = C.c_void_p, C.c_int, C.c_int64, C.c_float, C.c_double
        L.oracle_first_reject.restype = C.c_int32
        L.oracle_first_reject.argtypes = [vp, i32]
        L.oracle_softmax_stats.restype = None
        L.oracle_softmax_stats.argtypes = [vp, i32, i32, vp, vp]
        L.oracle_softmax_probs.restype = None
        L.oracle_softmax_probs.argtypes = [vp, i32, i32, vp]
        L.oracle_inverse_cdf.restype = C.c_int32
        L.oracle_inverse_cdf.argtypes = [vp, i32, f64]
        L.oracle_sample_softmax_row.restype = C.c_int32
        L.oracle_sample_softmax_row.argtypes = [vp, i32, i32, f64]
        L.oracle_residual_weights.restype = f64
        L.oracle_residual_weights.argtypes = [vp, vp, i32, i32, vp]
        L.oracle_sprinter_verify.restype = i32
        L.oracle_sprinter_verify.argtypes = [vp, vp, vp, vp, vp, f32, i32, i32, i32, i32, i32,
                                             vp, vp, vp]
        L.oracle_replace_sample.restype = i32
        L.oracle_replace_sample.argtypes = [vp, i64, i32, i64, vp, vp, i32, i32, i32, vp, i32, vp]
        L.oracle_sd_verify.restype = i32
        L.oracle_sd_verify.argtypes = [vp, vp, i64, vp, vp, i32, i32, i32, i32, i32,
                                       vp, vp, vp, vp, vp, vp]
        L.oracle_cdf_margin.restype = f64
        L.oracle_cdf_margin.argtypes = [vp, i32, f64, vp]
        L.oracle_softmax_draw_margin.restype = f64
        L.oracle_softmax_draw_margin.argtypes = [vp, i32, i32, f64, vp]
        L.oracle_residual_draw_margin.restype = f64
        L.oracle_residual_draw_margin.argtypes = [vp, vp, i32, i32, f64, vp]
        L.oracle_philox4x32_10.restype = None
        L.oracle_philox4x32_10.argtypes = [vp, vp, vp]
        L.oracle_simulate_runs.restype = i32
        L.oracle_simulate_runs.argtypes = [C.c_uint64, i64, i64, i32, f32, f32, i32, vp, vp]
        _lib = L
    return _lib


def _dt(a: np.ndarray) -> int:
    if a.dtype == np.float32:
        return 0
    if a.dtype == np.uint16:
        return 1
    if a.dtype == np.float64:
        return 2
    raise TypeError(f"unsupported element type {a.dtype}")


def _c(a, dtype=None):
    a = np.ascontiguousarray(a) if dtype is None else np.ascontiguousarray(a, dtype=dtype)
    return a


def _p(a):
    return None if a is None else a.ctypes.data_as(C.c_void_p)


def first_reject(accept_row) -> int:
    a = _c(accept_row, np.uint8)
    return int(lib().oracle_first_reject(_p(a), a.shape[0]))


def softmax_stats(row):
    row = _c(row)
    mx, Z = C.c_double(), C.c_double()
    lib().oracle_softmax_stats(_p(row), _dt(row), row.shape[0], C.byref(mx), C.byref(Z))
    return mx.value, Z.value


def softmax_probs(row) -> np.ndarray:
    row = _c(row)
    out = np.empty(row.shape[0], np.float64)
    lib().oracle_softmax_probs(_p(row), _dt(row), row.shape[0], _p(out))
    return out


def inverse_cdf(w, u: float) -> int:
    w = _c(w, np.float64)
    return int(lib().oracle_inverse_cdf(_p(w), w.shape[0], float(u)))


def sample_softmax_row(row, u: float) -> int:
    row = _c(row)
    return int(lib().oracle_sample_softmax_row(_p(row), _dt(row), row.shape[0], float(u)))


def residual_weights(p_row, q_row):
    p_row, q_row = _c(p_row), _c(q_row)
    assert p_row.dtype == q_row.dtype and p_row.shape == q_row.shape
    w = np.empty(p_row.shape[0], np.float64)
    R = lib().oracle_residual_weights(_p(p_row), _p(q_row), _dt(p_row), p_row.shape[0], _p(w))
    return w, float(R)


def sprinter_verify(hidden, W1, b1, W2, b2, threshold: float):
    """hidden [B,K,d]; W1 [h,d] (or [d] for the single linear layer, with b1 = W2 = None).

    Returns (scores float64 [B,K], accept uint8 [B,K], first_reject int32 [B])."""
    hidden, W1 = _c(hidden), _c(W1)
    B, K, d = hidden.shape
    h = 0 if W1.ndim == 1 else W1.shape[0]
    assert W1.shape[-1] == d and W1.dtype == hidden.dtype
    b2 = _c(np.asarray(b2, np.float32).reshape(1))
    if h:
        b1 = _c(b1, np.float32)
        W2 = _c(W2)
        assert W2.dtype == hidden.dtype and W2.shape == (h,) and b1.shape == (h,)
    else:
        b1 = W2 = None
    scores = np.empty((B, K), np.float64)
    accept = np.empty((B, K), np.uint8)
    fr = np.empty((B,), np.int32)
    rc = lib().oracle_sprinter_verify(_p(hidden), _p(W1), _p(b1), _p(W2), _p(b2),
                                      float(threshold), B, K, d, h, _dt(hidden),
                                      _p(scores), _p(accept), _p(fr))
    if rc != OK:
        raise ValueError(f"oracle_sprinter_verify: error {rc}")
    return scores, accept, fr


def replace_sample(target_logits, V: int, uniforms, rows=None, first_reject=None, K: int = 0,
                   seq_stride: int = 1, return_status: bool = False):
    """target_logits [R, ldv]; returns tokens int32 [n] (n = len(uniforms))."""
    tl = _c(target_logits)
    assert tl.ndim == 2
    R, ldv = tl.shape
    u = _c(uniforms, np.float32)
    n = u.shape[0]
    rows = None if rows is None else _c(rows, np.int32)
    fr = None if first_reject is None else _c(first_reject, np.int32)
    tokens = np.empty((n,), np.int32)
    rc = lib().oracle_replace_sample(_p(tl), ldv, V, R, _p(rows), _p(fr), K, seq_stride, n,
                                     _p(u), _dt(tl), _p(tokens))
    if rc == ERR_ARG:
        raise ValueError("oracle_replace_sample: invalid argument")
    return (tokens, rc) if return_status else tokens


def sd_verify(p_logits, q_logits, V: int, draft_tokens, uniforms, return_status: bool = False):
    """p_logits [B,Kp,ldv], q_logits [B,K,ldv], draft_tokens [B,K], uniforms [B,K+1].

    Returns dict(accepted_len, correction_token, accept, p_tok, q_tok, residual_mass)."""
    p, q = _c(p_logits), _c(q_logits)
    assert p.dtype == q.dtype and p.ndim == 3 and q.ndim == 3
    B, Kp, ldv = p.shape
    K = q.shape[1]
    assert q.shape[0] == B and q.shape[2] == ldv
    x = _c(draft_tokens, np.int32)
    u = _c(uniforms, np.float32)
    assert x.shape == (B, K) and u.shape == (B, K + 1)
    out = dict(
        accepted_len=np.empty((B,), np.int32),
        correction_token=np.empty((B,), np.int32),
        accept=np.empty((B, K), np.uint8),
        p_tok=np.empty((B, K), np.float64),
        q_tok=np.empty((B, K), np.float64),
        residual_mass=np.empty((B,), np.float64),
    )
    rc = lib().oracle_sd_verify(_p(p), _p(q), ldv, _p(x), _p(u), B, K, Kp, V, _dt(p),
                                _p(out["accepted_len"]), _p(out["correction_token"]),
                                _p(out["accept"]), _p(out["p_tok"]), _p(out["q_tok"]),
                                _p(out["residual_mass"]))
    if rc == ERR_ARG:
        raise ValueError("oracle_sd_verify: invalid argument")
    return (out, rc) if return_status else out


def cdf_margin(w, u: float):
    w = _c(w, np.float64)
    t = C.c_int32()
    m = lib().oracle_cdf_margin(_p(w), w.shape[0], float(u), C.byref(t))
    return float(m), int(t.value)


def softmax_draw_margin(row, u: float):
    row = _c(row)
    t = C.c_int32()
    m = lib().oracle_softmax_draw_margin(_p(row), _dt(row), row.shape[0], float(u), C.byref(t))
    return float(m), int(t.value)


def residual_draw_margin(p_row, q_row, u: float):
    p_row, q_row = _c(p_row), _c(q_row)
    t = C.c_int32()
    m = lib().oracle_residual_draw_margin(_p(p_row), _p(q_row), _dt(p_row), p_row.shape[0],
                                          float(u), C.byref(t))
    return float(m), int(t.value)


def philox4x32_10(counter, key) -> np.ndarray:
    c = _c(counter, np.uint32)
    k = _c(key, np.uint32)
    assert c.shape == (4,) and k.shape == (2,)
    out = np.empty(4, np.uint32)
    lib().oracle_philox4x32_10(_p(c), _p(k), _p(out))
    return out


def simulate_runs(seed: int, runs: int, r: int, eta_tp: float, eta_fp: float, max_tokens: int,
                  first_run: int = 0):
    """Returns (n_accepted int32 [runs], histogram uint64 [max_tokens + 1])."""
    n = np.empty((runs,), np.int32)
    hist = np.empty((max_tokens + 1,), np.uint64)
    rc = lib().oracle_simulate_runs(int(seed), int(first_run), int(runs), int(r), float(eta_tp),
                                    float(eta_fp), int(max_tokens), _p(n), _p(hist))
    if rc != OK:
        raise ValueError(f"oracle_simulate_runs: error {rc}")
    return n, hist
