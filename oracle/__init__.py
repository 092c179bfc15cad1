"""ctypes loader for the CPU oracle (test infrastructure, never on the product path).

The oracle itself is ``pyramidsd_oracle.cpp``: plain double-precision C++ written from the paper
(Sec. 3.1-3.4, Fig. 1). This module only compiles it with ``g++ -O2`` and marshals numpy arrays.
Nothing here imports the CUDA package.
"""
from __future__ import annotations

import ctypes as C
import os
import subprocess

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "pyramidsd_oracle.cpp")
_LIB = os.path.join(_HERE, "libpsd_oracle.so")

F32, BF16, F64 = 0, 1, 2
FUZZY, STRICT, FUZZY_SD_FALLBACK, ASSISTED = 0, 1, 2, 3
JS, TV, KL = 0, 1, 2
FLAG_SMALL_NONFINITE, FLAG_LARGE_NONFINITE, FLAG_TOKEN_RANGE = 1, 2, 4

_lib = None


def build(force: bool = False) -> str:
    """Compile the oracle into a shared object next to its source (no CUDA involved)."""
    if force or not os.path.exists(_LIB) or os.path.getmtime(_LIB) < os.path.getmtime(_SRC):
        tmp = _LIB + f".tmp{os.getpid()}"
        subprocess.check_call(["g++", "-O2", "-std=c++17", "-fPIC", "-shared", "-pthread", _SRC, "-o", tmp])
        os.replace(tmp, _LIB)
    return _LIB


def lib():
    global _lib
    if _lib is None:
        _lib = C.CDLL(build())
        _lib.psd_oracle_divergence.restype = C.c_double
        _lib.psd_oracle_residual_mass.restype = C.c_double
        _lib.psd_oracle_bonus_uniform.restype = C.c_double
    return _lib


def _ptr(a):
    return None if a is None else a.ctypes.data_as(C.c_void_p)


def _as_logits(a):
    """Accept float32 / float64 arrays, or uint16 arrays holding bf16 bit patterns."""
    a = np.ascontiguousarray(a)
    if a.dtype == np.float32:
        return a, F32
    if a.dtype == np.float64:
        return a, F64
    if a.dtype == np.uint16:
        return a, BF16
    raise TypeError(f"logits dtype {a.dtype}: want float32, float64 or uint16 (bf16 bits)")


def philox4x32_10(ctr, key):
    c = np.asarray(ctr, dtype=np.uint32)
    k = np.asarray(key, dtype=np.uint32)
    out = np.zeros(4, dtype=np.uint32)
    lib().psd_oracle_philox4x32_10(_ptr(c), _ptr(k), _ptr(out))
    return out


def row_uniforms(seed: int, offset: int, row: int):
    u, u2 = C.c_double(), C.c_double()
    lib().psd_oracle_row_uniforms(C.c_uint64(seed), C.c_uint64(offset), C.c_uint32(row), C.byref(u), C.byref(u2))
    return u.value, u2.value


def softmax(logits, inv_temperature: float = 1.0):
    a, dt = _as_logits(np.asarray(logits).reshape(-1))
    p = np.zeros(a.shape[0], dtype=np.float64)
    ok = lib().psd_oracle_softmax(_ptr(a), dt, a.shape[0], C.c_double(inv_temperature), _ptr(p))
    return p, bool(ok)


def divergence(p_large, p_small, kind: int = JS) -> float:
    p = np.ascontiguousarray(p_large, dtype=np.float64)
    q = np.ascontiguousarray(p_small, dtype=np.float64)
    return lib().psd_oracle_divergence(_ptr(p), _ptr(q), p.shape[0], kind)


def residual_mass(p_large, p_small) -> float:
    p = np.ascontiguousarray(p_large, dtype=np.float64)
    q = np.ascontiguousarray(p_small, dtype=np.float64)
    return lib().psd_oracle_residual_mass(_ptr(p), _ptr(q), p.shape[0])


def inverse_cdf(w, u2: float) -> int:
    w = np.ascontiguousarray(w, dtype=np.float64)
    return lib().psd_oracle_inverse_cdf(_ptr(w), w.shape[0], C.c_double(u2))


def prefix_length(accept, n_valid: int) -> int:
    a = np.ascontiguousarray(accept, dtype=np.int32)
    return lib().psd_oracle_prefix_length(_ptr(a), n_valid)


def verify_stage(logits_small, logits_large, tokens, tau, mode=FUZZY, seed=0, offset=0, n_valid=None,
                 inv_temperature=1.0, div_kind=JS, n_threads=1, seq_ids=None):
    """One verification stage on host arrays shaped [B, K, V] (tokens [B, K]). Returns a dict.

    ``seq_ids`` (optional, [B]) gives each sequence's index in the full batch when the arrays are a
    sample of it, so that row (b, k) draws the Philox block of row ``seq_ids[b] * K + k``."""
    s, dt = _as_logits(logits_small)
    l, dt2 = _as_logits(logits_large)
    assert dt == dt2 and s.shape == l.shape and s.ndim == 3
    B, K, V = s.shape
    t = np.ascontiguousarray(tokens, dtype=np.int32).reshape(B, K)
    nv = None if n_valid is None else np.ascontiguousarray(n_valid, dtype=np.int32)
    ids = None if seq_ids is None else np.ascontiguousarray(seq_ids, dtype=np.int32)
    out = {
        "accept_len": np.zeros(B, np.int32), "next_token": np.zeros(B, np.int32),
        "div": np.zeros((B, K)), "p_small_tok": np.zeros((B, K)), "p_large_tok": np.zeros((B, K)),
        "resid_mass": np.zeros((B, K)), "row_flags": np.zeros((B, K), np.int32),
        "accept_bits": np.zeros((B, K), np.int32),
    }
    rc = lib().psd_oracle_verify_stage(
        _ptr(s), _ptr(l), _ptr(t), B, K, V, dt, C.c_int64(V), C.c_int64(V),
        C.c_double(float(tau)), int(mode), C.c_uint64(seed), C.c_uint64(offset), _ptr(nv),
        C.c_double(inv_temperature), int(div_kind), _ptr(ids),
        _ptr(out["accept_len"]), _ptr(out["next_token"]), _ptr(out["div"]), _ptr(out["p_small_tok"]),
        _ptr(out["p_large_tok"]), _ptr(out["resid_mass"]), _ptr(out["row_flags"]), _ptr(out["accept_bits"]),
        int(n_threads))
    if rc:
        raise ValueError(f"oracle verify_stage rc={rc}")
    return out


def verify(logits_draft, logits_qual, logits_target, draft_tokens, tau_q, tau_t, mode=FUZZY, seed=0, offset=0,
           inv_temperature=1.0, div_kind=JS, n_threads=1, seq_ids=None, mode_t=None):
    """Two-stage pyramid on host arrays: draft/qual [B, K_d, V], target [B, K_q, V]. ``mode`` is the
    qualifier stage's acceptance mode and ``mode_t`` the target stage's (default: the same); the assisted
    variant of Sec. 3.4 is ``mode=ASSISTED, mode_t=FUZZY``."""
    d, dt = _as_logits(logits_draft)
    q, dtq = _as_logits(logits_qual)
    t, dtt = _as_logits(logits_target)
    assert dt == dtq == dtt and d.shape == q.shape
    B, K_d, V = d.shape
    K_q = t.shape[1]
    tok = np.ascontiguousarray(draft_tokens, dtype=np.int32).reshape(B, K_d)
    ids = None if seq_ids is None else np.ascontiguousarray(seq_ids, dtype=np.int32)
    out = {
        "accept_len_q": np.zeros(B, np.int32), "next_token_q": np.zeros(B, np.int32),
        "accept_len": np.zeros(B, np.int32), "next_token": np.zeros(B, np.int32),
        "window": np.zeros((B, K_q), np.int32), "n_window": np.zeros(B, np.int32),
        "div_q": np.zeros((B, K_d)), "div_t": np.zeros((B, K_q)),
    }
    rc = lib().psd_oracle_verify(
        _ptr(d), _ptr(q), _ptr(t), _ptr(tok), B, K_d, K_q, V, dt,
        C.c_double(float(tau_q)), C.c_double(float(tau_t)), int(mode), int(mode if mode_t is None else mode_t),
        C.c_uint64(seed), C.c_uint64(offset),
        C.c_double(inv_temperature), int(div_kind), _ptr(ids),
        _ptr(out["accept_len_q"]), _ptr(out["next_token_q"]), _ptr(out["accept_len"]), _ptr(out["next_token"]),
        _ptr(out["window"]), _ptr(out["n_window"]), _ptr(out["div_q"]), _ptr(out["div_t"]), int(n_threads))
    if rc:
        raise ValueError(f"oracle verify rc={rc}")
    return out


def bonus_uniform(seed, offset, b):
    """The uniform behind sequence b's bonus draw: Philox counter (b, 1, offset_lo, offset_hi), output word 1."""
    return float(lib().psd_oracle_bonus_uniform(C.c_uint64(seed), C.c_uint64(offset), C.c_uint32(b)))


def verify_stage_bonus(logits_small, logits_large_k1, tokens, tau, mode=FUZZY, seed=0, offset=0, n_valid=None,
                       inv_temperature=1.0, div_kind=JS, n_threads=1, seq_ids=None):
    """One stage whose larger model supplies K+1 rows per sequence: small [B, K, V], large [B, K+1, V]. When
    every valid position is accepted, ``next_token`` is drawn from the large model's row after the last
    valid position (the bonus token) instead of being -1."""
    s, dt = _as_logits(logits_small)
    l, dt2 = _as_logits(logits_large_k1)
    B, K, V = s.shape
    assert dt == dt2 and l.shape == (B, K + 1, V)
    t = np.ascontiguousarray(tokens, dtype=np.int32).reshape(B, K)
    nv = None if n_valid is None else np.ascontiguousarray(n_valid, dtype=np.int32)
    ids = None if seq_ids is None else np.ascontiguousarray(seq_ids, dtype=np.int32)
    out = {"accept_len": np.zeros(B, np.int32), "next_token": np.zeros(B, np.int32), "div": np.zeros((B, K))}
    rc = lib().psd_oracle_verify_stage_bonus(
        _ptr(s), _ptr(l), _ptr(t), B, K, V, dt, C.c_double(float(tau)), int(mode), C.c_uint64(seed),
        C.c_uint64(offset), _ptr(nv), C.c_double(inv_temperature), int(div_kind), _ptr(ids),
        _ptr(out["accept_len"]), _ptr(out["next_token"]), _ptr(out["div"]), int(n_threads))
    if rc:
        raise ValueError(f"oracle verify_stage_bonus rc={rc}")
    return out


def verify_bonus(logits_draft, logits_qual, logits_target_k1, draft_tokens, tau_q, tau_t, mode=FUZZY, seed=0,
                 offset=0, n_threads=1, seq_ids=None, mode_t=None):
    """Two-stage pyramid whose target supplies K_q+1 rows per sequence: stage 1 and the window as in
    ``verify``; stage 2 is ``verify_stage_bonus`` on the window (Philox offset + 1)."""
    t, _ = _as_logits(logits_target_k1)
    q, _ = _as_logits(logits_qual)
    K_q = t.shape[1] - 1
    base = verify(logits_draft, logits_qual, np.ascontiguousarray(t[:, :K_q]), draft_tokens, tau_q, tau_t, mode, seed,
                  offset, n_threads=n_threads, seq_ids=seq_ids, mode_t=mode_t)
    s2 = verify_stage_bonus(np.ascontiguousarray(q[:, :K_q]), t, base["window"], tau_t, mode if mode_t is None else mode_t,
                            seed, offset + 1,
                            n_valid=base["n_window"], n_threads=n_threads, seq_ids=seq_ids)
    assert np.array_equal(s2["accept_len"], base["accept_len"])
    out = dict(base)
    out["next_token"] = s2["next_token"]
    return out


def lmhead_logits(hidden_bf16, W_bf16, n_threads=1):
    """hidden [M, d], W [d, V] as uint16 bf16 bit patterns -> double logits [M, V]."""
    h = np.ascontiguousarray(hidden_bf16, dtype=np.uint16)
    w = np.ascontiguousarray(W_bf16, dtype=np.uint16)
    M, d = h.shape
    V = w.shape[1]
    out = np.zeros((M, V), dtype=np.float64)
    lib().psd_oracle_lmhead_logits(_ptr(h), _ptr(w), M, d, V, _ptr(out), int(n_threads))
    return out


def verify_stage_mixed(logits_small, logits_large, tokens, tau, mode=FUZZY, seed=0, offset=0, div_kind=JS,
                       n_threads=1):
    """Single stage whose two logits tensors have different element types (fused LM-head variant)."""
    s, dts = _as_logits(logits_small)
    l, dtl = _as_logits(logits_large)
    B, K, V = s.shape
    t = np.ascontiguousarray(tokens, dtype=np.int32).reshape(B, K)
    out = {"accept_len": np.zeros(B, np.int32), "next_token": np.zeros(B, np.int32),
           "div": np.zeros((B, K)), "resid_mass": np.zeros((B, K))}
    rc = lib().psd_oracle_verify_stage_mixed(
        _ptr(s), dts, _ptr(l), dtl, _ptr(t), B, K, V, C.c_double(float(tau)), int(mode),
        C.c_uint64(seed), C.c_uint64(offset), int(div_kind),
        _ptr(out["accept_len"]), _ptr(out["next_token"]), _ptr(out["div"]), _ptr(out["resid_mass"]), int(n_threads))
    if rc:
        raise ValueError(f"oracle verify_stage_mixed rc={rc}")
    return out
