"""Thin ctypes binding over the C ABI declared in ``include/pyramidsd.h``.

Argument marshalling only: every function takes torch tensors (device memory) or plain ints/floats,
checks dtype / contiguity, and passes raw pointers to the entry point of the same name. There is no
Python or CPU implementation behind these calls; if the shared library is missing they raise.
"""
from __future__ import annotations

import ctypes as C
import os
from typing import Optional

import torch

from .build import LIB_PATH

F32, BF16 = 0, 1
FUZZY, STRICT, FUZZY_SD_FALLBACK, ASSISTED = 0, 1, 2, 3
DIV_JS, DIV_TV, DIV_KL = 0, 1, 2
KERNEL_AUTO, KERNEL_BASELINE, KERNEL_CLUSTER, KERNEL_CLUSTER_STREAMED = 0, 1, 2, 3
LMHEAD_TILES_AUTO, LMHEAD_TILES_ONE_SM = 0, 1
OK, ERR_INVALID_ARG, ERR_UNSUPPORTED, ERR_WORKSPACE, ERR_CUDA, ERR_TIMEOUT = 0, -1, -2, -3, -4, -5

EXPORTS = (
    "pyramidsd_verify_stage", "pyramidsd_verify_stage_ex", "pyramidsd_verify", "pyramidsd_verify_ex", "pyramidsd_verify_bonus",
    "pyramidsd_verify_host", "pyramidsd_pyramid_workspace_bytes", "pyramidsd_selftest_wait_timeout", "pyramidsd_release_stream",
    "pyramidsd_verify_stage_noalloc", "pyramidsd_verify_fused_lmhead", "pyramidsd_verify_fused_lmhead_ex",
    "pyramidsd_model_sd_throughput", "pyramidsd_model_psd_throughput", "pyramidsd_set_two_stage_policy",
    "pyramidsd_row_uniforms", "pyramidsd_workspace_bytes", "pyramidsd_set_stream", "pyramidsd_last_status", "pyramidsd_launch_count",
    "pyramidsd_kernel_timing_begin", "pyramidsd_kernel_timing_end",
    "pyramidsd_cluster_occupancy", "pyramidsd_version", "pyramidsd_status_string",
)


class StageArgs(C.Structure):
    """Mirror of ``psd_stage_args``."""
    _fields_ = [
        ("struct_size", C.c_uint32), ("dtype", C.c_int32),
        ("logits_small", C.c_void_p), ("logits_large", C.c_void_p), ("tokens", C.c_void_p),
        ("B", C.c_int32), ("K", C.c_int32), ("V", C.c_int32),
        ("mode", C.c_int32), ("div_kind", C.c_int32),
        ("threshold", C.c_float), ("inv_temperature", C.c_float),
        ("seq_stride_small", C.c_int64), ("seq_stride_large", C.c_int64),
        ("philox_seed", C.c_uint64), ("philox_offset", C.c_uint64),
        ("n_valid", C.c_void_p),
        ("out_accept_len", C.c_void_p), ("out_next_token", C.c_void_p),
        ("out_div", C.c_void_p), ("out_p_small_tok", C.c_void_p), ("out_p_large_tok", C.c_void_p),
        ("out_resid_mass", C.c_void_p), ("out_row_flags", C.c_void_p),
        ("workspace", C.c_void_p), ("workspace_bytes", C.c_size_t),
        ("stream", C.c_void_p), ("use_stream_field", C.c_int32), ("kernel_variant", C.c_int32),
        ("cluster_size", C.c_int32), ("large_has_bonus_row", C.c_int32),
        ("reserved0", C.c_int32), ("seq_index_base", C.c_int64),
    ]


class PyramidArgs(C.Structure):
    """Mirror of ``psd_pyramid_args``."""
    _fields_ = [
        ("struct_size", C.c_uint32), ("dtype", C.c_int32),
        ("logits_draft", C.c_void_p), ("logits_qual", C.c_void_p), ("logits_target", C.c_void_p),
        ("draft_tokens", C.c_void_p),
        ("B", C.c_int32), ("K_d", C.c_int32), ("K_q", C.c_int32), ("V", C.c_int32),
        ("mode_q", C.c_int32), ("mode_t", C.c_int32),
        ("tau_q", C.c_float), ("tau_t", C.c_float),
        ("inv_temperature", C.c_float), ("div_kind", C.c_int32),
        ("philox_seed", C.c_uint64), ("philox_offset", C.c_uint64),
        ("seq_index_base", C.c_int64),
        ("target_has_bonus_row", C.c_int32), ("schedule", C.c_int32),
        ("out_accept_len_q", C.c_void_p), ("out_next_token_q", C.c_void_p),
        ("out_accept_len", C.c_void_p), ("out_next_token", C.c_void_p),
        ("out_div_q", C.c_void_p), ("out_resid_q", C.c_void_p), ("out_div_t", C.c_void_p), ("out_resid_t", C.c_void_p),
        ("out_window", C.c_void_p), ("out_n_window", C.c_void_p),
        ("workspace", C.c_void_p), ("workspace_bytes", C.c_size_t),
        ("stream", C.c_void_p), ("use_stream_field", C.c_int32), ("kernel_variant", C.c_int32),
    ]


class LmheadArgs(C.Structure):
    """Mirror of ``psd_lmhead_args``."""
    _fields_ = [
        ("struct_size", C.c_uint32), ("mode", C.c_int32),
        ("hidden", C.c_void_p), ("w_t", C.c_void_p), ("logits_small", C.c_void_p), ("tokens", C.c_void_p),
        ("B", C.c_int32), ("K", C.c_int32), ("d_model", C.c_int32), ("V", C.c_int32),
        ("threshold", C.c_float), ("tile_variant", C.c_int32),
        ("div_kind", C.c_int32), ("reserved0", C.c_int32),
        ("philox_seed", C.c_uint64), ("philox_offset", C.c_uint64),
        ("seq_index_base", C.c_int64),
        ("out_accept_len", C.c_void_p), ("out_next_token", C.c_void_p),
        ("out_div", C.c_void_p), ("out_resid_mass", C.c_void_p),
        ("stream", C.c_void_p),
    ]


class PyramidSDError(RuntimeError):
    def __init__(self, status: int, where: str):
        self.status = status
        super().__init__(f"{where}: {status_string(status)} ({status})")


_lib = None


def load_library(path: Optional[str] = None):
    """dlopen the in-tree shared library (no build, no fallback)."""
    global _lib
    if _lib is not None and path is None:
        return _lib
    p = path or os.environ.get("PYRAMIDSD_LIB") or LIB_PATH   # PYRAMIDSD_LIB: another build of the same library
    if not os.path.exists(p):
        raise ImportError(f"{p} is missing: build it with `python -m paper_2510_12966_b200.build` "
                          "(there is no CPU fallback for the verification path)")
    lib = C.CDLL(p)
    i32, u64, f32, vp = C.c_int, C.c_uint64, C.c_float, C.c_void_p
    lib.pyramidsd_verify_stage.argtypes = [vp, vp, vp, i32, i32, i32, i32, f32, i32, u64, u64, vp, vp]
    lib.pyramidsd_verify_stage.restype = i32
    lib.pyramidsd_verify_stage_noalloc.argtypes = [vp, vp, vp, i32, i32, i32, i32, f32, i32, u64, u64, vp, vp, vp, vp]
    lib.pyramidsd_verify_stage_noalloc.restype = i32
    lib.pyramidsd_verify_fused_lmhead.argtypes = [vp, vp, vp, vp, i32, i32, i32, i32, f32, i32, u64, u64, vp, vp, vp, vp, vp]
    lib.pyramidsd_verify_fused_lmhead.restype = i32
    lib.pyramidsd_model_sd_throughput.argtypes = [C.c_double] * 4
    lib.pyramidsd_model_sd_throughput.restype = C.c_double
    lib.pyramidsd_model_psd_throughput.argtypes = [C.c_double] * 7
    lib.pyramidsd_model_psd_throughput.restype = C.c_double
    lib.pyramidsd_verify_stage_ex.argtypes = [C.POINTER(StageArgs)]
    lib.pyramidsd_verify_stage_ex.restype = i32
    lib.pyramidsd_verify_ex.argtypes = [C.POINTER(PyramidArgs)]
    lib.pyramidsd_verify_ex.restype = i32
    lib.pyramidsd_verify_fused_lmhead_ex.argtypes = [C.POINTER(LmheadArgs)]
    lib.pyramidsd_verify_fused_lmhead_ex.restype = i32
    lib.pyramidsd_pyramid_workspace_bytes.argtypes = [i32, i32, i32, i32, i32]
    lib.pyramidsd_pyramid_workspace_bytes.restype = C.c_size_t
    lib.pyramidsd_release_stream.argtypes = [vp]
    lib.pyramidsd_release_stream.restype = i32
    lib.pyramidsd_selftest_wait_timeout.argtypes = [vp]
    lib.pyramidsd_selftest_wait_timeout.restype = i32
    pyr = [vp, vp, vp, vp, i32, i32, i32, i32, i32, f32, f32, i32, u64, u64, vp, vp, vp, vp]
    lib.pyramidsd_verify.argtypes = pyr
    lib.pyramidsd_verify_bonus.restype = C.c_int
    lib.pyramidsd_verify_bonus.argtypes = pyr
    lib.pyramidsd_verify.restype = i32
    lib.pyramidsd_verify_host.argtypes = pyr
    lib.pyramidsd_verify_host.restype = i32
    lib.pyramidsd_row_uniforms.argtypes = [u64, u64, i32, vp, vp]
    lib.pyramidsd_row_uniforms.restype = i32
    lib.pyramidsd_workspace_bytes.argtypes = [i32, i32, i32, i32]
    lib.pyramidsd_workspace_bytes.restype = C.c_size_t
    lib.pyramidsd_set_two_stage_policy.argtypes = [i32]
    lib.pyramidsd_set_two_stage_policy.restype = i32
    lib.pyramidsd_set_stream.argtypes = [vp]
    lib.pyramidsd_set_stream.restype = i32
    lib.pyramidsd_last_status.argtypes = []
    lib.pyramidsd_last_status.restype = i32
    lib.pyramidsd_kernel_timing_begin.argtypes = []
    lib.pyramidsd_kernel_timing_begin.restype = i32
    lib.pyramidsd_kernel_timing_end.argtypes = [C.POINTER(C.c_double), C.POINTER(i32), C.POINTER(C.c_double), C.POINTER(i32)]
    lib.pyramidsd_kernel_timing_end.restype = i32
    lib.pyramidsd_launch_count.argtypes = []
    lib.pyramidsd_launch_count.restype = u64
    lib.pyramidsd_cluster_occupancy.argtypes = [i32, i32, i32, i32, C.POINTER(i32), C.POINTER(i32)]
    lib.pyramidsd_cluster_occupancy.restype = i32
    lib.pyramidsd_version.restype = C.c_char_p
    lib.pyramidsd_status_string.argtypes = [i32]
    lib.pyramidsd_status_string.restype = C.c_char_p
    if path is None:
        _lib = lib
    return lib


def status_string(status: int) -> str:
    return load_library().pyramidsd_status_string(int(status)).decode()


def version() -> str:
    return load_library().pyramidsd_version().decode()


def _check(rc: int, where: str):
    if rc != OK:
        raise PyramidSDError(rc, where)


def dtype_code(t: torch.Tensor) -> int:
    if t.dtype == torch.float32:
        return F32
    if t.dtype == torch.bfloat16:
        return BF16
    raise TypeError(f"logits dtype {t.dtype}: want float32 or bfloat16")


def _dev_ptr(t: Optional[torch.Tensor], dtype=None, name="tensor") -> Optional[int]:
    if t is None:
        return None
    if not t.is_cuda:
        raise ValueError(f"{name} must live in device memory")
    if not t.is_contiguous():
        raise ValueError(f"{name} must be contiguous")
    if dtype is not None and t.dtype != dtype:
        raise TypeError(f"{name} must be {dtype}, got {t.dtype}")
    return t.data_ptr()


def set_stream(stream: Optional[torch.cuda.Stream] = None) -> None:
    """Use ``stream`` (default: torch's current stream) for the entry points without a stream argument."""
    s = torch.cuda.current_stream() if stream is None else stream
    _check(load_library().pyramidsd_set_stream(C.c_void_p(s.cuda_stream)), "pyramidsd_set_stream")


TWO_STAGE_DEFAULT, TWO_STAGE_FUSED, TWO_STAGE_SEPARATE, TWO_STAGE_AUTO, TWO_STAGE_FUSED_ROWS = 0, 1, 2, 3, 4


def set_two_stage_policy(policy: int) -> None:
    """``pyramidsd_set_two_stage_policy``: one statistics launch for both stages (row pairs or row triples),
    stage by stage, or chosen per call (the default)."""
    _check(load_library().pyramidsd_set_two_stage_policy(int(policy)), "pyramidsd_set_two_stage_policy")


def last_status() -> int:
    return load_library().pyramidsd_last_status()


def release_stream(stream) -> None:
    """``pyramidsd_release_stream``: free the library-owned scratch of a stream before destroying it."""
    _check(load_library().pyramidsd_release_stream(C.c_void_p(stream.cuda_stream)), "pyramidsd_release_stream")


def selftest_wait_timeout(stream=None) -> int:
    """``pyramidsd_selftest_wait_timeout``: one kernel whose bounded wait runs out on purpose."""
    s = torch.cuda.current_stream() if stream is None else stream
    return load_library().pyramidsd_selftest_wait_timeout(C.c_void_p(s.cuda_stream))


def pyramid_workspace_bytes(B: int, K_d: int, K_q: int, V: int, dtype: int) -> int:
    return int(load_library().pyramidsd_pyramid_workspace_bytes(B, K_d, K_q, V, dtype))


def launch_count() -> int:
    return int(load_library().pyramidsd_launch_count())


def kernel_timing_begin() -> None:
    _check(load_library().pyramidsd_kernel_timing_begin(), "pyramidsd_kernel_timing_begin")


def kernel_timing_end():
    """Returns (ms_rowstats, n_rowstats, ms_finalize, n_finalize) accumulated since kernel_timing_begin()."""
    a, b, c, d = C.c_double(0), C.c_int(0), C.c_double(0), C.c_int(0)
    _check(load_library().pyramidsd_kernel_timing_end(C.byref(a), C.byref(b), C.byref(c), C.byref(d)),
           "pyramidsd_kernel_timing_end")
    return a.value, b.value, c.value, d.value


def workspace_bytes(B: int, K: int, V: int, dtype: int) -> int:
    return int(load_library().pyramidsd_workspace_bytes(B, K, V, dtype))


def cluster_occupancy(B: int, K: int, V: int, dtype: int):
    """(cluster size, co-resident clusters) the library uses for this stage shape; (0, 0) = baseline kernel."""
    cs, n = C.c_int(0), C.c_int(0)
    _check(load_library().pyramidsd_cluster_occupancy(B, K, V, dtype, C.byref(cs), C.byref(n)), "pyramidsd_cluster_occupancy")
    return cs.value, n.value


def row_uniforms(philox_seed: int, offset: int, n_rows: int, device="cuda"):
    """``pyramidsd_row_uniforms``: the (u, u2) pair of every row as two float32 device tensors."""
    u = torch.empty(n_rows, dtype=torch.float32, device=device)
    u2 = torch.empty(n_rows, dtype=torch.float32, device=device)
    _check(load_library().pyramidsd_row_uniforms(int(philox_seed), int(offset), n_rows, u.data_ptr(), u2.data_ptr()),
           "pyramidsd_row_uniforms")
    return u, u2


def verify_stage(logits_small, logits_large, draft_tokens, threshold, mode=FUZZY, philox_seed=0, offset=0,
                 out_accept_len=None, out_next_token=None):
    """``pyramidsd_verify_stage`` on [B, K, V] device tensors; returns (accept_len [B], next_token [B])."""
    B, K, V = logits_small.shape
    dt = dtype_code(logits_small)
    assert logits_large.shape == logits_small.shape and logits_large.dtype == logits_small.dtype
    dev = logits_small.device
    if out_accept_len is None:
        out_accept_len = torch.empty(B, dtype=torch.int32, device=dev)
    if out_next_token is None:
        out_next_token = torch.empty(B, dtype=torch.int32, device=dev)
    rc = load_library().pyramidsd_verify_stage(
        _dev_ptr(logits_small, name="logits_small"), _dev_ptr(logits_large, name="logits_large"),
        _dev_ptr(draft_tokens, torch.int32, "draft_tokens"), B, K, V, dt, float(threshold), int(mode),
        int(philox_seed), int(offset), _dev_ptr(out_accept_len, torch.int32), _dev_ptr(out_next_token, torch.int32))
    _check(rc, "pyramidsd_verify_stage")
    return out_accept_len, out_next_token


def verify_fused_lmhead(hidden, w_t, logits_small, tokens, threshold, mode=FUZZY, philox_seed=0, offset=0, *,
                        want_rows=True, stream=None, raise_on_error=True, tile_variant=None, seq_index_base=0,
                        div_kind=DIV_JS, want_resid=None):
    """``pyramidsd_verify_fused_lmhead``: hidden [B*K, d] bf16, w_t [V, d] bf16 (LM-head weight, out x in),
    logits_small [B, K, V] bf16, tokens [B, K]. Returns a dict of device tensors (+ "status")."""
    B, K, V = logits_small.shape
    d = hidden.shape[1]
    assert hidden.shape[0] == B * K and w_t.shape == (V, d)
    dev = hidden.device
    out = {"accept_len": torch.empty(B, dtype=torch.int32, device=dev),
           "next_token": torch.empty(B, dtype=torch.int32, device=dev)}
    want_resid = want_rows if want_resid is None else want_resid
    if want_rows:
        out["div"] = torch.empty((B, K), dtype=torch.float32, device=dev)
    if want_resid:
        out["resid_mass"] = torch.empty((B, K), dtype=torch.float32, device=dev)
    s = torch.cuda.current_stream() if stream is None else stream
    if tile_variant is None and seq_index_base == 0 and div_kind == DIV_JS:
        rc = load_library().pyramidsd_verify_fused_lmhead(
            _dev_ptr(hidden, torch.bfloat16, "hidden"), _dev_ptr(w_t, torch.bfloat16, "w_t"),
            _dev_ptr(logits_small, torch.bfloat16, "logits_small"), _dev_ptr(tokens, torch.int32, "tokens"),
            B, K, d, V, float(threshold), int(mode), int(philox_seed), int(offset),
            out["accept_len"].data_ptr(), out["next_token"].data_ptr(),
            out["div"].data_ptr() if want_rows else None, out["resid_mass"].data_ptr() if want_resid else None,
            C.c_void_p(s.cuda_stream))
    else:
        a = LmheadArgs()
        a.struct_size = C.sizeof(LmheadArgs)
        a.mode = int(mode)
        a.hidden, a.w_t = _dev_ptr(hidden, torch.bfloat16, "hidden"), _dev_ptr(w_t, torch.bfloat16, "w_t")
        a.logits_small = _dev_ptr(logits_small, torch.bfloat16, "logits_small")
        a.tokens = _dev_ptr(tokens, torch.int32, "tokens")
        a.B, a.K, a.d_model, a.V = B, K, d, V
        a.threshold, a.tile_variant, a.div_kind = float(threshold), int(tile_variant or 0), int(div_kind)
        a.philox_seed, a.philox_offset, a.seq_index_base = int(philox_seed), int(offset), int(seq_index_base)
        a.out_accept_len, a.out_next_token = out["accept_len"].data_ptr(), out["next_token"].data_ptr()
        if want_rows:
            a.out_div = out["div"].data_ptr()
        if want_resid:
            a.out_resid_mass = out["resid_mass"].data_ptr()
        a.stream = s.cuda_stream
        rc = load_library().pyramidsd_verify_fused_lmhead_ex(C.byref(a))
    out["status"] = rc
    if raise_on_error:
        _check(rc, "pyramidsd_verify_fused_lmhead")
    return out


def model_sd_throughput(beta, ell, v_small, v_large) -> float:
    """Sec. 3.3: tokens/s of (fuzzy) speculative decoding for one model pair."""
    return load_library().pyramidsd_model_sd_throughput(beta, ell, v_small, v_large)


def model_psd_throughput(beta_qd, ell_d, v_draft, v_qual, beta_tq, ell_q, v_target) -> float:
    """Sec. 3.3: tokens/s of the three-model pyramid."""
    return load_library().pyramidsd_model_psd_throughput(beta_qd, ell_d, v_draft, v_qual, beta_tq, ell_q, v_target)


NOALLOC_MAX_ROWS = 8192


def verify_stage_noalloc(logits_small, logits_large, draft_tokens, threshold, mode=FUZZY, philox_seed=0, offset=0, *,
                         out_accept_len, out_next_token, out_wait_timeout=None, stream=None, raise_on_error=True):
    """``pyramidsd_verify_stage_noalloc``: the single stage with its scratch inside the library image, for
    callers that may not allocate device memory. Every output tensor is the caller's (this wrapper
    creates none); B * K is limited to NOALLOC_MAX_ROWS. Returns the status code."""
    B, K, V = logits_small.shape
    s = torch.cuda.current_stream() if stream is None else stream
    rc = load_library().pyramidsd_verify_stage_noalloc(
        _dev_ptr(logits_small, name="logits_small"), _dev_ptr(logits_large, name="logits_large"),
        _dev_ptr(draft_tokens, torch.int32, "draft_tokens"), B, K, V, dtype_code(logits_small), float(threshold),
        int(mode), int(philox_seed), int(offset), _dev_ptr(out_accept_len, torch.int32),
        _dev_ptr(out_next_token, torch.int32), _dev_ptr(out_wait_timeout, torch.int32), C.c_void_p(s.cuda_stream))
    if raise_on_error:
        _check(rc, "pyramidsd_verify_stage_noalloc")
    return rc


def verify_stage_ex(logits_small, logits_large, tokens, threshold, mode=FUZZY, philox_seed=0, offset=0, *,
                    B=None, K=None, V=None, n_valid=None, inv_temperature=0.0, div_kind=DIV_JS,
                    seq_stride_small=0, seq_stride_large=0, want_rows=True, workspace=None, stream=None,
                    kernel_variant=KERNEL_AUTO, cluster_size=0, raise_on_error=True, large_has_bonus_row=False,
                    seq_index_base=0, want_resid=None):
    """``pyramidsd_verify_stage_ex``: every option exposed. Returns a dict of device tensors (+ "status").
    With ``large_has_bonus_row`` the large logits are [B, K + 1, V]. ``want_resid`` (default: as ``want_rows``) asks
    for the rows' residual masses; without them the KL divergence takes the one-pass statistics kernel."""
    if B is None:
        B, K, V = logits_small.shape
        assert tuple(logits_large.shape) == (B, K + (1 if large_has_bonus_row else 0), V)
    dt = dtype_code(logits_small)
    dev = logits_small.device
    out = {"accept_len": torch.empty(B, dtype=torch.int32, device=dev),
           "next_token": torch.empty(B, dtype=torch.int32, device=dev)}
    want_resid = want_rows if want_resid is None else (want_resid and want_rows)
    if want_rows:
        for k in ("div", "p_small_tok", "p_large_tok") + (("resid_mass",) if want_resid else ()):
            out[k] = torch.empty((B, K), dtype=torch.float32, device=dev)
        out["row_flags"] = torch.empty((B, K), dtype=torch.int32, device=dev)
    a = StageArgs()
    a.struct_size = C.sizeof(StageArgs)
    a.dtype = dt
    a.logits_small = logits_small.data_ptr()
    a.logits_large = logits_large.data_ptr()
    a.tokens = _dev_ptr(tokens, torch.int32, "tokens")
    a.B, a.K, a.V = B, K, V
    a.mode, a.div_kind = int(mode), int(div_kind)
    a.threshold, a.inv_temperature = float(threshold), float(inv_temperature)
    a.seq_stride_small, a.seq_stride_large = int(seq_stride_small), int(seq_stride_large)
    a.philox_seed, a.philox_offset = int(philox_seed), int(offset)
    a.n_valid = _dev_ptr(n_valid, torch.int32, "n_valid")
    a.out_accept_len = out["accept_len"].data_ptr()
    a.out_next_token = out["next_token"].data_ptr()
    if want_rows:
        a.out_div = out["div"].data_ptr()
        a.out_p_small_tok = out["p_small_tok"].data_ptr()
        a.out_p_large_tok = out["p_large_tok"].data_ptr()
        if want_resid:
            a.out_resid_mass = out["resid_mass"].data_ptr()
        a.out_row_flags = out["row_flags"].data_ptr()
    if workspace is not None:
        a.workspace = workspace.data_ptr()
        a.workspace_bytes = workspace.numel() * workspace.element_size()
    s = torch.cuda.current_stream() if stream is None else stream
    a.stream = s.cuda_stream
    a.use_stream_field = 1
    a.kernel_variant = int(kernel_variant)
    a.cluster_size = int(cluster_size)
    a.large_has_bonus_row = 1 if large_has_bonus_row else 0
    a.seq_index_base = int(seq_index_base)
    rc = load_library().pyramidsd_verify_stage_ex(C.byref(a))
    out["status"] = rc
    if raise_on_error:
        _check(rc, "pyramidsd_verify_stage_ex")
    return out


def verify(logits_draft, logits_qual, logits_target, draft_tokens, tau_q, tau_t, mode=FUZZY, philox_seed=0,
           offset=0, out=None):
    """``pyramidsd_verify`` (two-stage pyramid) on device tensors. Returns a dict of four [B] int32 tensors."""
    B, K_d, V = logits_draft.shape
    K_q = logits_target.shape[1]
    dt = dtype_code(logits_draft)
    assert logits_qual.shape == logits_draft.shape and logits_target.shape == (B, K_q, V)
    dev = logits_draft.device
    if out is None:
        out = {k: torch.empty(B, dtype=torch.int32, device=dev)
               for k in ("accept_len_q", "next_token_q", "accept_len", "next_token")}
    rc = load_library().pyramidsd_verify(
        _dev_ptr(logits_draft, name="logits_draft"), _dev_ptr(logits_qual, name="logits_qual"),
        _dev_ptr(logits_target, name="logits_target"), _dev_ptr(draft_tokens, torch.int32, "draft_tokens"),
        B, K_d, K_q, V, dt, float(tau_q), float(tau_t), int(mode), int(philox_seed), int(offset),
        out["accept_len_q"].data_ptr(), out["next_token_q"].data_ptr(),
        out["accept_len"].data_ptr(), out["next_token"].data_ptr())
    _check(rc, "pyramidsd_verify")
    return out


def verify_ex(logits_draft, logits_qual, logits_target, draft_tokens, tau_q, tau_t, mode_q=FUZZY, mode_t=None,
              philox_seed=0, offset=0, *, seq_index_base=0, target_has_bonus_row=False, schedule=TWO_STAGE_DEFAULT,
              inv_temperature=0.0, div_kind=DIV_JS, want_rows=True, want_window=True, workspace=None, stream=None,
              kernel_variant=KERNEL_AUTO, raise_on_error=True, out=None, want_resid=None):
    """``pyramidsd_verify_ex``: the two-stage pyramid with per-stage modes, a sequence base, per-row outputs, the
    window, a caller workspace and an explicit schedule. Returns a dict of device tensors (+ "status"). ``out`` may
    bring the four [B] int32 result tensors (keys accept_len_q, next_token_q, accept_len, next_token)."""
    B, K_d, V = logits_draft.shape
    K_q = logits_target.shape[1] - (1 if target_has_bonus_row else 0)
    assert logits_qual.shape == logits_draft.shape and logits_target.shape[0] == B and logits_target.shape[2] == V
    dev = logits_draft.device
    if out is None:
        out = {k: torch.empty(B, dtype=torch.int32, device=dev)
               for k in ("accept_len_q", "next_token_q", "accept_len", "next_token")}
    else:
        out = dict(out)
    a = PyramidArgs()
    a.struct_size = C.sizeof(PyramidArgs)
    a.dtype = dtype_code(logits_draft)
    a.logits_draft = _dev_ptr(logits_draft, name="logits_draft")
    a.logits_qual = _dev_ptr(logits_qual, logits_draft.dtype, "logits_qual")
    a.logits_target = _dev_ptr(logits_target, logits_draft.dtype, "logits_target")
    a.draft_tokens = _dev_ptr(draft_tokens, torch.int32, "draft_tokens")
    a.B, a.K_d, a.K_q, a.V = B, K_d, K_q, V
    a.mode_q, a.mode_t = int(mode_q), int(mode_q if mode_t is None else mode_t)
    a.tau_q, a.tau_t = float(tau_q), float(tau_t)
    a.inv_temperature, a.div_kind = float(inv_temperature), int(div_kind)
    a.philox_seed, a.philox_offset, a.seq_index_base = int(philox_seed), int(offset), int(seq_index_base)
    a.target_has_bonus_row, a.schedule = (1 if target_has_bonus_row else 0), int(schedule)
    for k in ("accept_len_q", "next_token_q", "accept_len", "next_token"):
        setattr(a, "out_" + k, _dev_ptr(out[k], torch.int32, k))
    want_resid = want_rows if want_resid is None else (want_resid and want_rows)
    if want_rows:
        for k, n in (("div_q", K_d), ("resid_q", K_d), ("div_t", K_q), ("resid_t", K_q)):
            if k.startswith("resid") and not want_resid:
                continue   # without residual masses the KL divergence takes the one-pass statistics kernel
            out[k] = torch.empty((B, n), dtype=torch.float32, device=dev)
            setattr(a, "out_" + k, out[k].data_ptr())
    if want_window:
        out["window"] = torch.empty((B, K_q), dtype=torch.int32, device=dev)
        out["n_window"] = torch.empty(B, dtype=torch.int32, device=dev)
        a.out_window, a.out_n_window = out["window"].data_ptr(), out["n_window"].data_ptr()
    if workspace is not None:
        a.workspace = workspace.data_ptr()
        a.workspace_bytes = workspace.numel() * workspace.element_size()
    s = torch.cuda.current_stream() if stream is None else stream
    a.stream, a.use_stream_field = s.cuda_stream, 1
    a.kernel_variant = int(kernel_variant)
    rc = load_library().pyramidsd_verify_ex(C.byref(a))
    out["status"] = rc
    if raise_on_error:
        _check(rc, "pyramidsd_verify_ex")
    return out


def verify_bonus(logits_draft, logits_qual, logits_target, draft_tokens, tau_q, tau_t, mode=FUZZY, philox_seed=0,
                 offset=0, out=None):
    """``pyramidsd_verify_bonus``: the two-stage pyramid with a target of K_q + 1 rows per sequence
    (``logits_target`` [B, K_q + 1, V]); fully accepted windows get the target's bonus token."""
    B, K_d, V = logits_draft.shape
    K_q = logits_target.shape[1] - 1
    dt = dtype_code(logits_draft)
    assert logits_qual.shape == logits_draft.shape and logits_target.shape == (B, K_q + 1, V)
    dev = logits_draft.device
    if out is None:
        out = {k: torch.empty(B, dtype=torch.int32, device=dev)
               for k in ("accept_len_q", "next_token_q", "accept_len", "next_token")}
    rc = load_library().pyramidsd_verify_bonus(
        _dev_ptr(logits_draft, name="logits_draft"), _dev_ptr(logits_qual, name="logits_qual"),
        _dev_ptr(logits_target, name="logits_target"), _dev_ptr(draft_tokens, torch.int32, "draft_tokens"),
        B, K_d, K_q, V, dt, float(tau_q), float(tau_t), int(mode), int(philox_seed), int(offset),
        out["accept_len_q"].data_ptr(), out["next_token_q"].data_ptr(),
        out["accept_len"].data_ptr(), out["next_token"].data_ptr())
    _check(rc, "pyramidsd_verify_bonus")
    return out


def verify_host(logits_draft, logits_qual, logits_target, draft_tokens, tau_q, tau_t, mode=FUZZY, philox_seed=0,
                offset=0, out=None):
    """``pyramidsd_verify_host``: all tensors are HOST tensors (pinned for speed); copies are inside the call."""
    B, K_d, V = logits_draft.shape
    K_q = logits_target.shape[1]
    dt = dtype_code(logits_draft)
    for t in (logits_draft, logits_qual, logits_target, draft_tokens):
        if t.is_cuda or not t.is_contiguous():
            raise ValueError("verify_host takes contiguous host tensors")
    if out is None:
        out = {k: torch.empty(B, dtype=torch.int32).pin_memory()
               for k in ("accept_len_q", "next_token_q", "accept_len", "next_token")}
    rc = load_library().pyramidsd_verify_host(
        logits_draft.data_ptr(), logits_qual.data_ptr(), logits_target.data_ptr(), draft_tokens.data_ptr(),
        B, K_d, K_q, V, dt, float(tau_q), float(tau_t), int(mode), int(philox_seed), int(offset),
        out["accept_len_q"].data_ptr(), out["next_token_q"].data_ptr(),
        out["accept_len"].data_ptr(), out["next_token"].data_ptr())
    _check(rc, "pyramidsd_verify_host")
    return out
