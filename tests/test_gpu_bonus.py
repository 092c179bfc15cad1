"""GPU parity for the bonus token: a window whose positions were all accepted ends with a token of the larger
model, drawn from the row after the window (Sec. 1; large logits [B, K + 1, V])."""
import numpy as np
import pytest
import torch

from parity_utils import TOL, compare_stage, dtype_name, gpu_stage_to_numpy, host_bits

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def psd():
    if not torch.cuda.is_available():
        pytest.skip("no CUDA device")
    from paper_2510_12966_b200 import binding
    binding.load_library()
    torch.cuda.set_device(0)
    return binding


@pytest.fixture(scope="module")
def wl():
    from paper_2510_12966_b200 import workloads
    return workloads


def check_bonus_tokens(oracle, gpu, orc, zl_host, nv, K, seed, offset, dtype, inv_temperature=1.0):
    """Sequences that both sides accepted in full: the bonus tokens agree, or differ only across an inverse-CDF
    boundary that lies within the tolerance class of the dtype. Returns (sequences checked, near ties)."""
    n, ties = 0, 0
    for b in range(len(nv)):
        if not (gpu["accept_len"][b] == nv[b] == orc["accept_len"][b]):
            continue
        n += 1
        tg, to = int(gpu["next_token"][b]), int(orc["next_token"][b])
        if tg == to:
            continue
        assert tg >= 0 and to >= 0, f"seq {b}: bonus token gpu {tg} oracle {to}"
        p, ok = oracle.softmax(zl_host[b, nv[b]], inv_temperature)
        assert ok and p[tg] > 0
        c = np.cumsum(p)
        target = oracle.bonus_uniform(seed, offset, b) * c[-1]
        lo, hi = min(tg, to), max(tg, to)
        between = c[hi - 1] - c[lo] if hi - 1 > lo else 0.0
        assert abs(c[lo] - target) / c[-1] < TOL[dtype]["cdf"] and between / c[-1] < TOL[dtype]["cdf"], \
            f"seq {b}: bonus token gpu {tg} oracle {to} is not a near tie"
        ties += 1
    return n, ties


def run_bonus_stage(psd, oracle, zs, zl1, tok, tau, mode=0, seed=0, offset=0, n_valid=None, variant=0):
    dev = torch.device("cuda:0")
    B, K, V = zs.shape
    nv_d = None if n_valid is None else torch.as_tensor(n_valid, dtype=torch.int32, device=dev)
    out = psd.verify_stage_ex(zs.to(dev), zl1.to(dev), tok.to(dev), tau, mode, seed, offset, n_valid=nv_d,
                              kernel_variant=variant, large_has_bonus_row=True)
    torch.cuda.synchronize()
    assert psd.last_status() == 0
    gpu = gpu_stage_to_numpy(out)
    zs_h, zl_h = host_bits(zs), host_bits(zl1)
    nv = np.full(B, K, np.int32) if n_valid is None else np.clip(np.asarray(n_valid, np.int32), 0, K)
    plain = oracle.verify_stage(zs_h, np.ascontiguousarray(zl_h[:, :K]), tok.numpy(), np.float32(tau), mode, seed, offset,
                                n_valid=n_valid, n_threads=8)
    bonus = oracle.verify_stage_bonus(zs_h, zl_h, tok.numpy(), np.float32(tau), mode, seed, offset, n_valid=n_valid,
                                      n_threads=8)
    # everything but the bonus draw is the plain stage: compare with the bonus tokens taken out
    full = gpu["accept_len"] == nv
    masked = dict(gpu)
    masked["next_token"] = np.where(full, -1, gpu["next_token"])
    rep = compare_stage(oracle, masked, plain, zs_h, np.ascontiguousarray(zl_h[:, :K]), dtype=dtype_name(zs), mode=mode,
                        tau=float(np.float32(tau)), seed=seed, offset=offset, n_valid=n_valid)
    n, ties = check_bonus_tokens(oracle, gpu, bonus, zl_h, nv, K, seed, offset, dtype_name(zs))
    return gpu, bonus, rep, n, ties


@pytest.mark.parametrize("dtype,V", [("bf16", 128256), ("f32", 32000), ("f32", 1001), ("bf16", 4099)])
def test_bonus_token_when_everything_is_accepted(psd, oracle, wl, dtype, V):
    """tau = 1 > ln 2 accepts every position; windows of every length, the empty one included (its bonus
    row is row 0). V = 1001 and 4099 take the scalar loads."""
    B, K = 7, 4
    zs, zl, tok = wl.make_stage_inputs(B, K + 1, V, dtype, seed=600 + V, sigma=0.8)
    zs = zs[:, :K].contiguous()
    tok = tok[:, :K].contiguous()
    nv = [0, 1, 2, 3, 4, 4, 4]
    gpu, orc, rep, n, ties = run_bonus_stage(psd, oracle, zs, zl, tok, 1.0, seed=5, offset=11, n_valid=nv)
    assert n == B and ties <= 1
    assert np.array_equal(gpu["accept_len"], nv) and np.all(gpu["next_token"] >= 0)
    gpu2, _, _, _, _ = run_bonus_stage(psd, oracle, zs, zl, tok, 1.0, seed=5, offset=12, n_valid=nv)
    assert not np.array_equal(gpu["next_token"], gpu2["next_token"])      # the offset moves the draw


@pytest.mark.parametrize("mode", [0, 1, 3])
def test_bonus_token_mixed_with_rejections(psd, oracle, wl, mode):
    B, K, V = 40, 3, 32768
    zs, zl, tok = wl.make_stage_inputs(B, K + 1, V, "bf16", seed=700 + mode, sigma=0.35, boost=(9.0, 12.0))
    zs = zs[:, :K].contiguous()
    tok = tok[:, :K].contiguous()
    probe = oracle.verify_stage(host_bits(zs), np.ascontiguousarray(host_bits(zl)[:, :K]), tok.numpy(), 1.0, 0, 0, 0, n_threads=8)
    tau = float(np.float32(np.quantile(probe["div"], 0.8)))
    gpu, orc, rep, n, ties = run_bonus_stage(psd, oracle, zs, zl, tok, tau, mode=mode, seed=3, offset=mode)
    assert n >= 3 and (mode != 0 or B - n >= 3), n   # fully accepted windows are present (and, by the threshold, others)
    assert rep["tie_div"] + rep["tie_coin"] + rep["tie_cdf"] + ties <= 2


def test_bonus_row_without_a_distribution(psd, oracle, wl):
    B, K, V = 4, 2, 8200
    zs, zl, tok = wl.make_stage_inputs(B, K + 1, V, "f32", seed=801, sigma=0.5)
    zs = zs[:, :K].contiguous()
    tok = tok[:, :K].contiguous()
    zl[0, K, 4000] = float("nan")
    zl[1, K, :] = -float("inf")
    zl[2, K, 17] = float("inf")
    zl[3, K, :5000] = -float("inf")                # masked vocabulary is fine
    gpu, orc, _, n, _ = run_bonus_stage(psd, oracle, zs, zl, tok, 1.0)
    assert n == B
    assert list(gpu["next_token"][:3]) == [-2, -2, -2] and gpu["next_token"][3] >= 5000
    assert np.array_equal(gpu["next_token"], orc["next_token"])


def test_bonus_token_window_of_32(psd, oracle, wl):
    B, K, V = 2, 32, 2048
    zs, zl, tok = wl.make_stage_inputs(B, K + 1, V, "f32", seed=802, sigma=0.5)
    zs = zs[:, :K].contiguous()
    tok = tok[:, :K].contiguous()
    gpu, orc, _, n, ties = run_bonus_stage(psd, oracle, zs, zl, tok, 1.0, seed=1, offset=1)
    assert n == B and ties == 0 and np.array_equal(gpu["accept_len"], [32, 32])


def test_stride_too_small_for_the_bonus_row_is_refused(psd, wl):
    dev = torch.device("cuda:0")
    zs, zl, tok = [t.to(dev) for t in wl.make_stage_inputs(2, 3, 4096, "f32", seed=803)]
    out = psd.verify_stage_ex(zs[:, :2].contiguous(), zl, tok[:, :2].contiguous(), 0.1, B=2, K=2, V=4096,
                              seq_stride_large=2 * 4096, large_has_bonus_row=True, raise_on_error=False)
    assert out["status"] == psd.ERR_INVALID_ARG


@pytest.mark.parametrize("mode", [0, 1])
@pytest.mark.parametrize("policy", ["fused", "separate"])
def test_pyramid_bonus_matches_oracle(psd, oracle, wl, mode, policy):
    """Two stages with a target of K_q + 1 rows: stage 1 and the window as without the bonus row; windows the
    target accepts in full end with the target's bonus token. Both schedules of the wrapper."""
    B, K_d, K_q, V = 24, 8, 4, 128256
    zd, zq, zt, tok = wl.make_pyramid_inputs(B, K_d, K_q + 1, V, "bf16", seed=900 + mode, sigma_q=0.25, sigma_d=0.5,
                                             boost=(9.0, 12.0))
    dev = torch.device("cuda:0")
    tau_q, tau_t = 0.0, 0.0
    if mode == 0:   # thresholds that let most windows through stage 1 and about half of them through stage 2
        probe = oracle.verify(host_bits(zd), host_bits(zq), np.ascontiguousarray(host_bits(zt)[:, :K_q]), tok.numpy(), 1.0, 1.0,
                              0, 7, 20, n_threads=8)
        tau_q = float(np.float32(np.quantile(probe["div_q"], 0.9)))
        tau_t = float(np.float32(np.quantile(probe["div_t"], 0.8)))
    try:
        psd.set_two_stage_policy(psd.TWO_STAGE_SEPARATE if policy == "separate" else psd.TWO_STAGE_FUSED)
        out = psd.verify_bonus(zd.to(dev), zq.to(dev), zt.to(dev), tok.to(dev), tau_q, tau_t, mode, 7, 20)
        torch.cuda.synchronize()
    finally:
        psd.set_two_stage_policy(psd.TWO_STAGE_DEFAULT)
    assert psd.last_status() == 0
    gpu = gpu_stage_to_numpy(out)
    zt_h = host_bits(zt)
    orc = oracle.verify_bonus(host_bits(zd), host_bits(zq), zt_h, tok.numpy(), np.float32(tau_q), np.float32(tau_t), mode, 7, 20,
                              n_threads=8)
    same = (gpu["accept_len_q"] == orc["accept_len_q"]) & (gpu["next_token_q"] == orc["next_token_q"]) & \
           (gpu["accept_len"] == orc["accept_len"])
    assert same.sum() >= B - 2                      # near ties upstream are rare
    full = same & (orc["accept_len"] == orc["n_window"])
    assert full.sum() >= 3 and (mode != 0 or B - full.sum() >= 3), full.sum()
    mism = 0
    for b in np.nonzero(same)[0]:
        if gpu["next_token"][b] != orc["next_token"][b]:
            mism += 1
    assert mism <= 1
    assert np.all(gpu["next_token"][full] >= 0)
