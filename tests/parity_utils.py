"""Comparison of the CUDA library's results with the CPU oracle's, with the counted near-tie classes.

Exactly one result is correct per seed. A disagreement in an integer output is tolerated only when the
oracle's own margin shows the decision was a near tie, and every such case is counted and reported:
  (i)   fuzzy accept:   |D - tau| < 1e-4;
  (ii)  coin flip:      |u - min(1, p_large(x)/p_small(x))| < tol_coin (1e-5 fp32, 2e-3 bf16);
  (iii) inverse CDF:    the oracle's target u' * W lies within tol_cdf * W of the prefix-sum boundary that
                        separates the two tokens (1e-6 fp32, 1e-4 bf16).
  (iv)  unresolved residual: the oracle's residual mass at the rejected row is below 1e-6 -- less than single
                        precision, in which the library takes sum max(p, q) - 1, can tell from zero. The library
                        then draws from p_large, as the rule for a zero residual says; its token must have
                        positive p_large.
A sequence whose accept length differs because of (i)/(ii) is not compared further.
Floating-point outputs (divergence, residual mass, token probabilities) must agree within `tol_val`:
1e-5 absolute with fp32 logits, 2e-3 absolute with bf16 logits.
"""
from __future__ import annotations

import numpy as np
import torch

TOL = {
    "f32": dict(val=1e-5, coin=1e-5, cdf=1e-6),
    "bf16": dict(val=2e-3, coin=2e-3, cdf=1e-4),
}
TIE_DIV = 1e-4
RESID_FLOOR = 1e-6


def dtype_name(t: torch.Tensor) -> str:
    return "f32" if t.dtype == torch.float32 else "bf16"


def host_bits(t: torch.Tensor) -> np.ndarray:
    t = t.detach().cpu().contiguous()
    if t.dtype == torch.bfloat16:
        return t.view(torch.int16).numpy().view(np.uint16)
    return t.numpy()


def compare_stage(oracle, gpu, orc, zs_host, zl_host, *, dtype, mode, tau, seed, offset, n_valid=None,
                  seq_ids=None, div_kind=0, inv_temperature=1.0, check_rows=True):
    """gpu: dict of numpy arrays from the library; orc: dict from oracle.verify_stage. Returns a report."""
    tol = TOL[dtype]
    B, K = orc["div"].shape
    nv = np.full(B, K, np.int32) if n_valid is None else np.clip(np.asarray(n_valid), 0, K)
    rep = dict(rows=int(nv.sum()), seqs=B, tie_div=0, tie_coin=0, tie_cdf=0, tie_resid=0, max_err_div=0.0, max_err_prob=0.0,
               max_err_resid=0.0)
    valid = np.arange(K)[None, :] < nv[:, None]
    ok_rows = valid & (orc["row_flags"] == 0)

    if check_rows and "div" in gpu:
        fin = ok_rows & np.isfinite(orc["div"])
        if fin.any():
            rep["max_err_div"] = float(np.abs(gpu["div"][fin] - orc["div"][fin]).max())
            if "resid_mass" in gpu:   # a caller may leave the residual masses out
                rep["max_err_resid"] = float(np.abs(gpu["resid_mass"][fin] - orc["resid_mass"][fin]).max())
            rep["max_err_prob"] = float(max(np.abs(gpu["p_small_tok"][ok_rows] - orc["p_small_tok"][ok_rows]).max(),
                                            np.abs(gpu["p_large_tok"][ok_rows] - orc["p_large_tok"][ok_rows]).max()))
        assert rep["max_err_div"] <= tol["val"], f"divergence error {rep['max_err_div']}"
        assert rep["max_err_resid"] <= tol["val"], f"residual-mass error {rep['max_err_resid']}"
        assert rep["max_err_prob"] <= tol["val"], f"token-probability error {rep['max_err_prob']}"
        inf_rows = ok_rows & np.isinf(orc["div"])
        assert np.all(np.isinf(gpu["div"][inf_rows]))
        nonfinite = 3  # flag bits 1 | 2
        assert np.array_equal(gpu["row_flags"][valid] != 0, orc["row_flags"][valid] != 0)
        assert np.array_equal(gpu["row_flags"][valid] & nonfinite, orc["row_flags"][valid] & nonfinite)

    for b in range(B):
        Lg, Lo = int(gpu["accept_len"][b]), int(orc["accept_len"][b])
        gid = b if seq_ids is None else int(seq_ids[b])
        if Lg != Lo:
            k = min(Lg, Lo)
            assert k < nv[b], f"seq {b}: accept_len gpu {Lg} oracle {Lo} beyond n_valid {nv[b]}"
            d = orc["div"][b, k]
            u, _ = oracle.row_uniforms(seed, offset, gid * K + k)
            pl, ps = orc["p_large_tok"][b, k], orc["p_small_tok"][b, k]
            rho = (pl / ps) if ps > 0 else (np.inf if pl > 0 else 0.0)
            tie_d = mode in (0, 2) and abs(d - tau) < TIE_DIV
            tie_c = mode in (1, 2, 3) and abs(u - min(1.0, rho)) < tol["coin"]
            assert tie_d or tie_c, (f"seq {b} pos {k}: accept_len gpu {Lg} oracle {Lo}, D={d} tau={tau} "
                                    f"u={u} rho={rho} — not a near tie")
            rep["tie_div" if tie_d else "tie_coin"] += 1
            continue
        tg, to = int(gpu["next_token"][b]), int(orc["next_token"][b])
        if tg == to:
            continue
        assert Lo < nv[b] and tg >= 0 and to >= 0, f"seq {b}: next_token gpu {tg} oracle {to}"
        # inverse-CDF near tie: rebuild the oracle's weights and prefix sums for row (b, Lo)
        p, _ = oracle.softmax(zl_host[b, Lo], inv_temperature)
        q, _ = oracle.softmax(zs_host[b, Lo], inv_temperature)
        w = np.maximum(p - q, 0.0)
        if mode != 3 and 0 < orc["resid_mass"][b, Lo] < RESID_FLOOR:
            assert p[tg] > 0, f"seq {b}: gpu token {tg} has zero probability under the large model"
            rep["tie_resid"] += 1
            continue
        if mode == 3 or not (orc["resid_mass"][b, Lo] > 0):
            w = p
        c = np.cumsum(w)
        _, u2 = oracle.row_uniforms(seed, offset, gid * K + Lo)
        target = u2 * c[-1]
        lo = min(tg, to)
        margin = abs(c[lo] - target) / c[-1]
        assert w[tg] > 0, f"seq {b}: gpu token {tg} has zero weight"
        between = c[max(tg, to) - 1] - c[lo] if max(tg, to) - 1 > lo else 0.0
        assert margin < tol["cdf"] and between / c[-1] < tol["cdf"], (
            f"seq {b} row {Lo}: token gpu {tg} oracle {to}, margin {margin:.3e} of W — not a near tie")
        rep["tie_cdf"] += 1
    return rep


def gpu_stage_to_numpy(out: dict) -> dict:
    return {k: (v.detach().cpu().numpy() if isinstance(v, torch.Tensor) else v) for k, v in out.items()}
