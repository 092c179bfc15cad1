"""GPU parity of the one-pass statistics kernel: with the KL(large || small) divergence, whose terms separate, and no
caller waiting for per-row residual masses, batches of at least one row per SM take both softmax normalisers and the
divergence in a single sweep over the logits. Element by element against the oracle (divergences, flags, accept
lengths, tokens), on masked, flagged and identical rows, on a row whose late logits overflow the running sums, with
ragged n_valid, and through every schedule of the two-stage call."""
import numpy as np
import pytest
import torch

from parity_utils import TOL, compare_stage, gpu_stage_to_numpy, host_bits

pytestmark = pytest.mark.gpu
KL = 2


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


def statistics_ms(psd, call):
    """Device time of the statistics launches of one call (the one-pass kernel shows as about half the two-pass time)."""
    psd.kernel_timing_begin()
    out = call()
    torch.cuda.synchronize()
    ms, n, _, _ = psd.kernel_timing_end()
    return out, ms, n


# the last two shapes give every CTA eight and four rows (the partial buffers and their barriers go round several times)
@pytest.mark.parametrize("dtype,V,B,K", [("f32", 4100, 40, 4), ("bf16", 8200, 30, 5), ("bf16", 50264, 20, 8), ("f32", 32000, 38, 4),
                                         ("bf16", 4096, 150, 8), ("f32", 6000, 100, 6)])
def test_one_pass_against_oracle(psd, oracle, wl, dtype, V, B, K):
    dev = torch.device("cuda:0")
    zs, zl, tok = wl.make_stage_inputs(B, K, V, dtype, seed=600 + V, sigma=0.6)
    zs[1, 0, 100:900] = -float("inf")          # the small model masks tokens the large one keeps: KL = +inf
    zl[2, 1, 200:300] = -float("inf")          # the other way round: those terms vanish
    zs[3, 0, 7] = float("nan")
    zl[4, 1, :] = zs[4, 1, :]                  # identical rows: exactly 0
    zl[5, 0, 3] = float("inf")
    zs[6, 1, :] = -float("inf")                # no finite logit
    zl[7, 0, :64] = -float("inf")              # rows that start with masked tokens
    zs[7, 0, :64] = -float("inf")
    n_valid = np.random.default_rng(V).integers(0, K + 1, size=B).astype(np.int32)
    n_valid[:10] = K
    d = [t.to(dev) for t in (zs, zl, tok)]
    nv_d = torch.as_tensor(n_valid, device=dev)
    assert B * K >= 148
    for tau, mode in ((0.05, 0), (0.3, 0), (0.05, 1), (0.05, 2), (0.0, 3)):
        out = psd.verify_stage_ex(*d, tau, mode, 3, 1, div_kind=KL, n_valid=nv_d, want_resid=False)
        torch.cuda.synchronize()
        assert psd.last_status() == 0 and "resid_mass" not in out
        gpu = gpu_stage_to_numpy(out)
        orc = oracle.verify_stage(host_bits(zs), host_bits(zl), tok.numpy(), np.float32(tau), mode, 3, 1, n_valid=n_valid,
                                  div_kind=KL, n_threads=8)
        rep = compare_stage(oracle, gpu, orc, host_bits(zs), host_bits(zl), dtype=dtype, mode=mode, tau=float(np.float32(tau)),
                            seed=3, offset=1, n_valid=n_valid, div_kind=KL)
        assert rep["tie_div"] + rep["tie_coin"] + rep["tie_cdf"] <= 2
        assert gpu["div"][4, 1] == 0.0 and np.isinf(gpu["div"][1, 0]) and gpu["row_flags"][3, 0] == 1
        assert gpu["row_flags"][5, 0] == 2 and gpu["row_flags"][6, 1] == 1
    # the same call with the residual masses asked for runs the two-pass kernel: same decisions, divergences within
    # the tolerance of each other
    two = gpu_stage_to_numpy(psd.verify_stage_ex(*d, 0.05, 0, 3, 1, div_kind=KL, n_valid=nv_d))
    one = gpu_stage_to_numpy(psd.verify_stage_ex(*d, 0.05, 0, 3, 1, div_kind=KL, n_valid=nv_d, want_resid=False))
    fin = np.isfinite(two["div"]) & (np.arange(K)[None, :] < n_valid[:, None])
    assert np.abs(two["div"][fin] - one["div"][fin]).max() <= 2 * TOL[dtype]["val"]
    assert np.array_equal(two["accept_len"], one["accept_len"])


def test_one_pass_is_the_kernel_that_runs(psd, wl):
    """Half the exps and one read instead of two: the statistics launch of a KL call without residual masses takes well
    under the time of the same call with them."""
    dev = torch.device("cuda:0")
    d = [t.to(dev) for t in wl.make_stage_inputs(64, 8, 65536, "bf16", seed=9, sigma=0.6)]
    for _ in range(2):
        psd.verify_stage_ex(*d, 0.1, 0, 0, 0, div_kind=KL)
        psd.verify_stage_ex(*d, 0.1, 0, 0, 0, div_kind=KL, want_resid=False)
    two = [statistics_ms(psd, lambda: psd.verify_stage_ex(*d, 0.1, 0, 0, 0, div_kind=KL)) for _ in range(5)]
    one = [statistics_ms(psd, lambda: psd.verify_stage_ex(*d, 0.1, 0, 0, 0, div_kind=KL, want_resid=False)) for _ in range(5)]
    assert all(n == 1 for _, _, n in two + one)
    ms_two, ms_one = min(ms for _, ms, _ in two), min(ms for _, ms, _ in one)      # the best of five: a shared GPU has hiccups
    assert ms_one < 0.75 * ms_two, (ms_one, ms_two)


def test_one_pass_late_logits_far_above_the_first_ones(psd, oracle, wl):
    """A warp takes its reference from its first vectors of a row; logits 200 nats above them overflow its running sums,
    and the warp goes over its share of the row again against the true maxima. The results are the oracle's."""
    dev = torch.device("cuda:0")
    B, K, V = 40, 4, 20000
    zs, zl, tok = wl.make_stage_inputs(B, K, V, "f32", seed=17, sigma=0.4)
    for b in range(0, B, 3):
        zs[b, 1, :4096] -= 150.0
        zl[b, 1, :4096] -= 150.0
        zs[b, 1, 9000:9100] += 60.0
        zl[b, 1, 9000:9100] += 60.5
    d = [t.to(dev) for t in (zs, zl, tok)]
    out = psd.verify_stage_ex(*d, 0.05, 0, 3, 1, div_kind=KL, want_resid=False)
    torch.cuda.synchronize()
    assert psd.last_status() == 0
    gpu = gpu_stage_to_numpy(out)
    orc = oracle.verify_stage(host_bits(zs), host_bits(zl), tok.numpy(), np.float32(0.05), 0, 3, 1, div_kind=KL, n_threads=8)
    rep = compare_stage(oracle, gpu, orc, host_bits(zs), host_bits(zl), dtype="f32", mode=0, tau=float(np.float32(0.05)), seed=3,
                        offset=1, div_kind=KL)
    assert rep["tie_div"] + rep["tie_cdf"] <= 2 and np.all(np.isfinite(gpu["div"]))


@pytest.mark.parametrize("dtype", ["bf16", "f32"])
def test_one_pass_in_every_schedule_of_the_two_stage_call(psd, oracle, wl, dtype):
    dev = torch.device("cuda:0")
    B, K_d, K_q, V = 24, 6, 4, 16384
    zd, zq, zt, tok = wl.make_pyramid_inputs(B, K_d, K_q, V, dtype, seed=33, sigma_q=0.3, sigma_d=0.6)
    dd = [t.to(dev) for t in (zd, zq, zt, tok)]
    probe = psd.verify_ex(*dd, 1e9, 1e9, div_kind=KL)
    tau_q, tau_t = float(probe["div_q"].median()), float(probe["div_t"].median())
    outs = []
    for schedule in (psd.TWO_STAGE_FUSED, psd.TWO_STAGE_SEPARATE, psd.TWO_STAGE_FUSED_ROWS, psd.TWO_STAGE_AUTO):
        o = psd.verify_ex(*dd, tau_q, tau_t, 0, 0, 5, 9, div_kind=KL, schedule=schedule, want_resid=False)
        torch.cuda.synchronize()
        assert psd.last_status() == 0 and "resid_q" not in o
        outs.append(o)
    for o in outs[1:]:
        for k in ("accept_len_q", "next_token_q", "accept_len", "next_token", "window", "n_window", "div_q"):
            x, y = outs[0][k], o[k]
            if x.dtype == torch.float32:
                x, y = x.view(torch.int32), y.view(torch.int32)
            assert torch.equal(x, y), k
        inside = torch.arange(K_q, device=dev)[None, :] < o["n_window"][:, None]
        assert torch.equal(outs[0]["div_t"].view(torch.int32)[inside], o["div_t"].view(torch.int32)[inside])
    gpu = gpu_stage_to_numpy(outs[0])
    orc = oracle.verify(host_bits(zd), host_bits(zq), host_bits(zt), tok.numpy(), np.float32(tau_q), np.float32(tau_t), 0, 5, 9,
                        div_kind=KL, n_threads=8)
    o1 = oracle.verify_stage(host_bits(zd), host_bits(zq), tok.numpy(), np.float32(tau_q), 0, 5, 9, div_kind=KL, n_threads=8)
    assert np.abs(gpu["div_q"] - o1["div"]).max() <= TOL[dtype]["val"]
    same = (gpu["accept_len_q"] == orc["accept_len_q"]) & (gpu["next_token_q"] == orc["next_token_q"])
    assert same.sum() >= B - 2
    assert np.array_equal(gpu["accept_len"][same], orc["accept_len"][same])
    assert (gpu["next_token"][same] == orc["next_token"][same]).sum() >= same.sum() - 1
    assert 0 < orc["accept_len_q"].sum() < B * K_d


@pytest.mark.parametrize("cfg", [3, 4])
def test_full_size_configs_with_kl_sampled(psd, oracle, wl, cfg):
    """The launch configurations `bench.py --div kl` times (config 3: B=64, V=128256, K=16/8; config 4: B=256, V=152064,
    K=8/4; bf16), checked on sampled sequences: the oracle runs them with their indices in the batch, so the coin flips
    and draws are those of the full call."""
    dev = torch.device("cuda:0")
    w = wl.CONFIGS[cfg]
    zd, zq, zt, tok = wl.workload_inputs(cfg, 0, device="cpu")
    dd = [t.to(dev) for t in (zd, zq, zt, tok)]
    probe = psd.verify_ex(*dd, 1e9, 1e9, div_kind=KL)
    tau_q, tau_t = float(probe["div_q"].median()), float(probe["div_t"].median())
    psd.kernel_timing_begin()
    out = psd.verify_ex(*dd, tau_q, tau_t, 0, 0, 0, 4, div_kind=KL, want_resid=False)
    torch.cuda.synchronize()
    ms, n, _, _ = psd.kernel_timing_end()
    assert psd.last_status() == 0 and n in (1, 2)      # one statistics launch, or two when the call runs stage by stage
    gpu = gpu_stage_to_numpy(out)
    ids = np.array([0, 17, 40, w.B - 1])
    sub = [host_bits(t[ids]) for t in (zd, zq, zt)]
    orc = oracle.verify(*sub, tok.numpy()[ids], np.float32(tau_q), np.float32(tau_t), 0, 0, 4, div_kind=KL, n_threads=8, seq_ids=ids)
    o1 = oracle.verify_stage(sub[0], sub[1], tok.numpy()[ids], np.float32(tau_q), 0, 0, 4, div_kind=KL, n_threads=8, seq_ids=ids)
    assert np.abs(gpu["div_q"][ids] - o1["div"]).max() <= TOL["bf16"]["val"]
    near = np.abs(o1["div"] - tau_q).min() < 1e-4
    if not near:
        assert np.array_equal(gpu["accept_len_q"][ids], orc["accept_len_q"])
        same = gpu["next_token_q"][ids] == orc["next_token_q"]
        assert same.sum() >= len(ids) - 1
        assert np.array_equal(gpu["accept_len"][ids][same], orc["accept_len"][same])
    assert 0 < gpu["accept_len_q"].sum() < w.B * w.K_d


def test_one_pass_draw_on_identical_rows(psd, oracle, wl):
    """The one-pass record carries no residual mass; a rejected row whose two distributions are identical (residual
    exactly zero) is found out by the draw itself, which then takes p_large as the oracle does."""
    dev = torch.device("cuda:0")
    B, K, V = 50, 3, 8192
    zs, zl, tok = wl.make_stage_inputs(B, K, V, "f32", seed=91, sigma=0.5)
    zl[::2] = zs[::2]                           # every other sequence: identical rows
    d = [t.to(dev) for t in (zs, zl, tok)]
    out = psd.verify_stage_ex(*d, -1.0, 0, 6, 2, div_kind=KL, want_resid=False)       # tau < 0: position 0 is rejected everywhere
    torch.cuda.synchronize()
    assert psd.last_status() == 0
    gpu = gpu_stage_to_numpy(out)
    orc = oracle.verify_stage(host_bits(zs), host_bits(zl), tok.numpy(), np.float32(-1.0), 0, 6, 2, div_kind=KL, n_threads=8)
    assert np.all(gpu["accept_len"] == 0) and np.all(gpu["next_token"] >= 0) and np.all(gpu["div"][::2] == 0.0)
    rep = compare_stage(oracle, gpu, orc, host_bits(zs), host_bits(zl), dtype="f32", mode=0, tau=-1.0, seed=6, offset=2, div_kind=KL)
    assert rep["tie_cdf"] <= 1 and rep["tie_div"] == 0
