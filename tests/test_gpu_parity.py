"""GPU parity: the CUDA library, called through its C ABI, against the CPU oracle on the same seeded
inputs and the same Philox stream. Sizes span several tiles and ragged tails; reduced versions of the
benchmark workloads run element by element, and the full-size bench configuration is checked on sampled
sequences."""
import math

import numpy as np
import pytest
import torch

from parity_utils import TOL, compare_stage, dtype_name, gpu_stage_to_numpy, host_bits

pytestmark = pytest.mark.gpu

LN2 = math.log(2.0)


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


def run_stage_both(psd, oracle, zs, zl, tok, tau, mode=0, seed=0, offset=0, n_valid=None, inv_temperature=0.0,
                   div_kind=0, variant=0, cluster_size=0):
    """Library on the GPU, oracle on the host, same bits. Returns (gpu dict, oracle dict, report)."""
    dev = torch.device("cuda:0")
    zs_d, zl_d, tok_d = zs.to(dev), zl.to(dev), tok.to(dev)
    nv_d = None if n_valid is None else torch.as_tensor(n_valid, dtype=torch.int32, device=dev)
    out = psd.verify_stage_ex(zs_d, zl_d, tok_d, tau, mode, seed, offset, n_valid=nv_d,
                              inv_temperature=inv_temperature, div_kind=div_kind, kernel_variant=variant,
                              cluster_size=cluster_size)
    torch.cuda.synchronize()
    assert psd.last_status() == 0
    gpu = gpu_stage_to_numpy(out)
    zs_h, zl_h = host_bits(zs), host_bits(zl)
    invT = inv_temperature if inv_temperature > 0 else 1.0
    orc = oracle.verify_stage(zs_h, zl_h, tok.numpy(), np.float32(tau), mode, seed, offset, n_valid=n_valid,
                              inv_temperature=float(np.float32(invT)), div_kind=div_kind, n_threads=8)
    rep = compare_stage(oracle, gpu, orc, zs_h, zl_h, dtype=dtype_name(zs), mode=mode, tau=float(np.float32(tau)),
                        seed=seed, offset=offset, n_valid=n_valid, div_kind=div_kind,
                        inv_temperature=float(np.float32(invT)))
    return gpu, orc, rep


# --------------------------------------------------------------------------------------------------
def test_row_uniforms_match_oracle_philox(psd, oracle):
    seed, offset, n = 0x9E3779B97F4A7C15, (1 << 40) + 12345, 100_000
    u, u2 = psd.row_uniforms(seed, offset, n)
    u, u2 = u.cpu().numpy(), u2.cpu().numpy()
    rows = np.r_[0:2000, n - 2000:n]
    for r in rows:
        a, b = oracle.row_uniforms(seed, offset, int(r))
        assert u[r] == np.float32(a) and u2[r] == np.float32(b)
    assert 0.0 <= u.min() and u.max() < 1.0


@pytest.mark.parametrize("dtype", ["f32", "bf16"])
@pytest.mark.parametrize("V", [5, 16, 17, 1000, 4099, 8192, 8200, 32000, 50257])
def test_stage_fuzzy_small_shapes(psd, oracle, wl, dtype, V):
    B, K = 3, 5
    zs, zl, tok = wl.make_stage_inputs(B, K, V, dtype, seed=100 + V, sigma=0.8)
    for tau in (0.02, 0.1, 0.3):
        _, _, rep = run_stage_both(psd, oracle, zs, zl, tok, tau, seed=V, offset=7)
        assert rep["tie_div"] + rep["tie_cdf"] <= 2


@pytest.mark.parametrize("dtype", ["f32", "bf16"])
@pytest.mark.parametrize("mode", [1, 2, 3])
def test_stage_coin_flip_modes(psd, oracle, wl, dtype, mode):
    B, K, V = 16, 6, 12000
    zs, zl, tok = wl.make_stage_inputs(B, K, V, dtype, seed=7, sigma=0.6)
    ties = 0
    for offset in range(4):
        _, orc, rep = run_stage_both(psd, oracle, zs, zl, tok, 0.05, mode=mode, seed=3, offset=offset)
        ties += rep["tie_coin"] + rep["tie_cdf"] + rep["tie_div"]
        assert 0 < orc["accept_len"].sum() < B * K   # the case exercises both outcomes
    assert ties <= 4


@pytest.mark.parametrize("div_kind", [1, 2])
def test_other_divergences(psd, oracle, wl, div_kind):
    zs, zl, tok = wl.make_stage_inputs(4, 4, 20000, "f32", seed=8, sigma=0.5)
    tau = 0.3 if div_kind == 1 else 0.5
    run_stage_both(psd, oracle, zs, zl, tok, tau, div_kind=div_kind)


def test_temperature(psd, oracle, wl):
    zs, zl, tok = wl.make_stage_inputs(4, 4, 20000, "f32", seed=9, sigma=0.5)
    run_stage_both(psd, oracle, zs, zl, tok, 0.2, inv_temperature=1 / 0.7)   # Sec. 4.1: temperature 0.7


def test_cfg1_tiny_fp32(psd, oracle, wl):
    """workload configuration 1: B=1, K=4, V=32000 fp32, fuzzy tau=0.3 and strict, Philox seed 0, several rounds."""
    ties = 0
    for rnd in range(8):
        zs, zl, tok = wl.workload_inputs(1, rnd)
        for mode in (0, 1):
            _, _, rep = run_stage_both(psd, oracle, zs, zl, tok, 0.3, mode=mode, seed=0, offset=rnd)
            ties += rep["tie_div"] + rep["tie_coin"] + rep["tie_cdf"]
            assert rep["max_err_div"] < 1e-5
    assert ties <= 1


def test_edge_identical_rows_and_thresholds(psd, oracle, wl):
    zs, zl, tok = wl.make_stage_inputs(2, 4, 5000, "bf16", seed=10)
    gpu, orc, _ = run_stage_both(psd, oracle, zl, zl, tok, 0.0)
    assert np.all(gpu["div"] == 0.0) and np.all(gpu["resid_mass"] == 0.0)
    assert np.all(gpu["accept_len"] == 4) and np.all(gpu["next_token"] == -1)
    gpu, _, _ = run_stage_both(psd, oracle, zs, zl, tok, np.float32(LN2) + 1e-6)   # tau >= max JS: all accepted
    assert np.all(gpu["accept_len"] == 4)
    gpu, _, _ = run_stage_both(psd, oracle, zs, zl, tok, -1e-6)                    # tau < 0: none accepted
    assert np.all(gpu["accept_len"] == 0) and np.all(gpu["next_token"] >= 0)
    # strict mode on identical rows: ratio 1, always accepted
    gpu, _, _ = run_stage_both(psd, oracle, zl, zl, tok, 0.0, mode=1)
    assert np.all(gpu["accept_len"] == 4)
    # disjoint supports: JS = ln 2, TV = 1
    z1 = torch.full((1, 1, 64), -float("inf"))
    z2 = z1.clone()
    z1[0, 0, 3] = 0.0
    z2[0, 0, 40] = 1.0
    gpu, orc, _ = run_stage_both(psd, oracle, z1, z2, torch.tensor([[3]], dtype=torch.int32), 0.5)
    assert abs(gpu["div"][0, 0] - LN2) < 1e-6 and abs(gpu["resid_mass"][0, 0] - 1.0) < 1e-6
    assert gpu["next_token"][0] == 40


def test_edge_masked_and_flagged_rows(psd, oracle, wl):
    zs, zl, tok = wl.make_stage_inputs(4, 3, 3000, "f32", seed=11, sigma=0.3)
    zs[0, 1, 100:900] = -float("inf")          # masked vocabulary on one side only
    zl[1, 0, :] = -float("inf")
    zl[1, 0, 5] = 2.0                           # a single live token
    zs[2, 1, 17] = float("nan")
    zl[3, 0, 2999] = float("inf")
    tok[0, 2] = 3000                             # out of range
    gpu, orc, _ = run_stage_both(psd, oracle, zs, zl, tok, 1.0)
    assert gpu["next_token"][2] == -2 and gpu["accept_len"][2] == 1
    assert gpu["next_token"][3] == -2 and gpu["accept_len"][3] == 0
    assert gpu["row_flags"][0, 2] == 4 and gpu["accept_len"][0] == 2
    zs2, zl2, tok2 = wl.make_stage_inputs(1, 2, 64, "f32", seed=12)
    zl2[0, 0, :] = -float("inf")                # a row with no finite entry is flagged too
    gpu, _, _ = run_stage_both(psd, oracle, zs2, zl2, tok2, 1.0)
    assert gpu["row_flags"][0, 0] == 2 and gpu["next_token"][0] == -2


def test_edge_empty_and_n_valid(psd, oracle, wl):
    dev = torch.device("cuda:0")
    zs, zl, tok = wl.make_stage_inputs(4, 6, 2048, "bf16", seed=13, sigma=0.2)
    gpu, orc, _ = run_stage_both(psd, oracle, zs, zl, tok, 0.5, n_valid=[0, 2, 6, 3])
    assert gpu["accept_len"][0] == 0 and gpu["next_token"][0] == -1
    empty = torch.empty((0, 6, 2048), dtype=torch.bfloat16, device=dev)
    out = psd.verify_stage_ex(empty, empty, torch.empty((0, 6), dtype=torch.int32, device=dev), 0.1)
    assert out["status"] == 0
    z0 = torch.empty((3, 0, 2048), dtype=torch.bfloat16, device=dev)
    out = psd.verify_stage_ex(z0, z0, torch.empty((3, 0), dtype=torch.int32, device=dev), 0.1, want_rows=False)
    torch.cuda.synchronize()
    assert out["accept_len"].tolist() == [0, 0, 0] and out["next_token"].tolist() == [-1, -1, -1]
    # K = 32, the widest window the scan takes
    zs, zl, tok = wl.make_stage_inputs(2, 32, 1024, "f32", seed=14, sigma=0.05)
    gpu, orc, _ = run_stage_both(psd, oracle, zs, zl, tok, 1.0)
    assert np.all(gpu["accept_len"] == 32)
    run_stage_both(psd, oracle, zs, zl, tok, 0.0005)


def test_bad_arguments_return_codes(psd, wl):
    dev = torch.device("cuda:0")
    zs, zl, tok = [t.to(dev) for t in wl.make_stage_inputs(1, 2, 64, "f32", seed=15)]
    assert psd.verify_stage_ex(zs, zl, tok, 0.1, mode=9, raise_on_error=False)["status"] == psd.ERR_INVALID_ARG
    assert psd.verify_stage_ex(zs, zl, tok, 0.1, div_kind=5, raise_on_error=False)["status"] == psd.ERR_INVALID_ARG
    assert psd.verify_stage_ex(zs, zl, tok, 0.1, K=33, B=1, V=64, raise_on_error=False)["status"] == psd.ERR_INVALID_ARG
    assert psd.verify_stage_ex(zs, zl, tok, float("nan"), raise_on_error=False)["status"] == psd.ERR_INVALID_ARG
    small_ws = torch.empty(256, dtype=torch.uint8, device=dev)
    assert psd.verify_stage_ex(zs, zl, tok, 0.1, workspace=small_ws, raise_on_error=False)["status"] == psd.ERR_WORKSPACE
    ws = torch.empty(psd.workspace_bytes(1, 2, 64, psd.F32), dtype=torch.uint8, device=dev)
    assert psd.verify_stage_ex(zs, zl, tok, 0.1, workspace=ws)["status"] == 0
    with pytest.raises(psd.PyramidSDError):
        psd.verify(zs, zs, zs, tok, 0.1, 0.1, mode=7)
    torch.cuda.synchronize()
    assert psd.last_status() == 0


def test_results_are_bit_identical_run_to_run(psd, wl):
    dev = torch.device("cuda:0")
    zs, zl, tok = [t.to(dev) for t in wl.make_stage_inputs(8, 8, 32000, "bf16", seed=16, sigma=0.7)]
    ref = None
    for _ in range(5):
        out = psd.verify_stage_ex(zs, zl, tok, 0.05, mode=2, philox_seed=1, offset=2)
        torch.cuda.synchronize()
        cur = {k: v.clone() for k, v in out.items() if isinstance(v, torch.Tensor)}
        if ref is not None:
            for k in ref:
                assert torch.equal(ref[k].view(torch.int32), cur[k].view(torch.int32)), k
        ref = cur


# -------------------------------------------------------------------------------------------------- cluster kernel
@pytest.mark.parametrize("dtype", ["f32", "bf16"])
@pytest.mark.parametrize("cs", [1, 2, 3, 4, 6, 8, 16])
@pytest.mark.parametrize("V", [2048, 8200, 32000, 128256])
def test_cluster_kernel_every_cluster_size(psd, oracle, wl, dtype, cs, V):
    """The cluster kernel with the cluster size forced: slices with ragged tails, empty slices (small V
    over many CTAs), one and several chunks per slice; a slice of more than 12 chunks does not fit the
    shared-memory ring and takes the streamed-twice variant (V = 128256 with one or two CTAs)."""
    B, K = 3, 5
    zs, zl, tok = wl.make_stage_inputs(B, K, V, dtype, seed=300 + V + cs, sigma=0.8)
    for tau in (0.02, 0.3):
        _, _, rep = run_stage_both(psd, oracle, zs, zl, tok, tau, seed=V, offset=cs, variant=psd.KERNEL_CLUSTER,
                                   cluster_size=cs)
        assert rep["tie_div"] + rep["tie_cdf"] <= 1


@pytest.mark.parametrize("dtype,V,B,K,cs", [("bf16", 32768, 48, 8, 1), ("f32", 16384, 40, 7, 0), ("bf16", 128256, 24, 16, 0),
                                            ("bf16", 128256, 24, 16, 4), ("bf16", 128256, 40, 16, 2), ("bf16", 128256, 50, 16, 1),
                                            ("f32", 65536, 60, 7, 1), ("f32", 152064, 24, 8, 2)])
def test_cluster_kernel_many_rows_per_cluster(psd, oracle, wl, dtype, V, B, K, cs):
    """More rows than resident clusters: every cluster walks several rows, so the ring(s), the exchange
    buffers and the barrier phases wrap around -- with the slice resident in the ring and, for the large
    vocabularies on one or two CTAs, streamed twice. Also checked against the baseline kernel."""
    zs, zl, tok = wl.make_stage_inputs(B, K, V, dtype, seed=400 + B, boost=(4.0, 12.0), sigma=0.7)
    nv = [(3 * b) % (K + 1) for b in range(B)]
    g1, orc, rep = run_stage_both(psd, oracle, zs, zl, tok, 0.15, mode=2, seed=4, offset=9, n_valid=nv,
                                  variant=psd.KERNEL_CLUSTER, cluster_size=cs)
    g2, _, _ = run_stage_both(psd, oracle, zs, zl, tok, 0.15, mode=2, seed=4, offset=9, n_valid=nv,
                              variant=psd.KERNEL_BASELINE)
    valid = np.arange(K)[None, :] < np.asarray(nv)[:, None]
    tol = TOL[dtype]["val"]
    assert np.abs(g1["div"][valid] - g2["div"][valid]).max() < tol
    assert np.abs(g1["resid_mass"][valid] - g2["resid_mass"][valid]).max() < tol
    assert rep["tie_div"] + rep["tie_coin"] + rep["tie_cdf"] <= 2


def test_cluster_kernel_masked_flagged_and_identical_rows(psd, oracle, wl):
    B, K, V = 4, 3, 16384
    zs, zl, tok = wl.make_stage_inputs(B, K, V, "bf16", seed=31, sigma=0.3)
    zs[0, 1, 100:9000] = -float("inf")          # masked vocabulary on one side, across a chunk boundary
    zl[1, 0, :] = -float("inf")
    zl[1, 0, 12345] = 2.0                        # a single live token
    zs[2, 1, 17] = float("nan")
    zl[3, 0, V - 1] = float("inf")
    zl[3, 2] = zs[3, 2]                          # bitwise identical pair
    zs[0, 0, :4096] = -3.0e38                    # huge negative finite logits
    for cs in (1, 2):
        gpu, orc, _ = run_stage_both(psd, oracle, zs, zl, tok, 1.0, variant=psd.KERNEL_CLUSTER, cluster_size=cs)
        assert gpu["next_token"][2] == -2 and gpu["accept_len"][2] == 1
        assert gpu["next_token"][3] == -2 and gpu["accept_len"][3] == 0
        assert gpu["next_token"][1] == 12345 or gpu["accept_len"][1] > 0
        assert np.all(np.isfinite(gpu["div"][0])) and np.all(np.isfinite(gpu["div"][1]))
    zs2, zl2, tok2 = wl.make_stage_inputs(1, 3, 4096, "f32", seed=32)
    zl2[0, 0, :] = -float("inf")                 # a row with no finite entry is flagged
    zl2[0, 2] = zs2[0, 2]
    gpu, _, _ = run_stage_both(psd, oracle, zs2, zl2, tok2, 1.0, variant=psd.KERNEL_CLUSTER, cluster_size=2)
    assert gpu["row_flags"][0, 0] == 2 and gpu["next_token"][0] == -2


def test_streamed_twice_masked_flagged_and_identical_rows(psd, oracle, wl):
    """The same edge rows where the slice does not fit the ring (V = 128256 on one or two CTAs): the careful
    second go of pass A then reads the row from global memory."""
    B, K, V = 4, 3, 128256
    zs, zl, tok = wl.make_stage_inputs(B, K, V, "bf16", seed=33, sigma=0.3)
    zs[0, 1, 100:90000] = -float("inf")          # masked vocabulary across many chunks
    zl[1, 0, :] = -float("inf")
    zl[1, 0, 101234] = 2.0                       # a single live token, late in the row
    zs[2, 1, 99999] = float("nan")
    zl[3, 0, V - 1] = float("inf")
    zl[3, 2] = zs[3, 2]                          # bitwise identical pair
    zs[0, 0, :70000] = -3.0e38                   # huge negative finite logits
    zl[0, 2, 120000] = 300.0                     # far above the row's first vectors: the optimistic sum overflows
    for cs in (1, 2):
        gpu, orc, _ = run_stage_both(psd, oracle, zs, zl, tok, 1.0, variant=psd.KERNEL_CLUSTER, cluster_size=cs)
        assert gpu["next_token"][2] == -2 and gpu["accept_len"][2] == 1
        assert gpu["next_token"][3] == -2 and gpu["accept_len"][3] == 0
        assert gpu["next_token"][1] == 101234 or gpu["accept_len"][1] > 0
        assert np.all(np.isfinite(gpu["div"][0])) and np.all(np.isfinite(gpu["div"][1]))


def test_streamed_twice_equals_resident_bit_for_bit(psd, wl):
    """PSD_KERNEL_CLUSTER_STREAMED makes a forced cluster size take the streamed-twice form also where the slice
    would fit the ring. Its arithmetic is the resident form's, so it must return the very same bits: one chunk and
    several per slice, ragged tails, more rows than clusters."""
    cases = [(7, 5, 2048, "f32", 1), (40, 8, 32768, "bf16", 1), (30, 8, 50000, "bf16", 2), (24, 16, 128256, "bf16", 4),
             (33, 7, 65536, "f32", 8)]
    dev = torch.device("cuda:0")
    for i, (B, K, V, dt, cs) in enumerate(cases):
        zs, zl, tok = [t.to(dev) for t in wl.make_stage_inputs(B, K, V, dt, seed=500 + i, sigma=0.7)]
        r = psd.verify_stage_ex(zs, zl, tok, 0.2, 2, 5, 6, kernel_variant=psd.KERNEL_CLUSTER, cluster_size=cs)
        q = psd.verify_stage_ex(zs, zl, tok, 0.2, 2, 5, 6, kernel_variant=psd.KERNEL_CLUSTER_STREAMED, cluster_size=cs)
        torch.cuda.synchronize()
        assert psd.last_status() == 0
        for k, v in r.items():
            if torch.is_tensor(v):
                assert torch.equal(v.view(torch.int32), q[k].view(torch.int32)), (i, k)
    bad = psd.verify_stage_ex(zs, zl, tok, 0.2, kernel_variant=psd.KERNEL_CLUSTER_STREAMED, raise_on_error=False)
    assert bad["status"] == psd.ERR_INVALID_ARG          # the streamed form wants an explicit cluster size


@pytest.mark.parametrize("div_kind", [1, 2])
def test_cluster_kernel_other_divergences(psd, oracle, wl, div_kind):
    zs, zl, tok = wl.make_stage_inputs(4, 4, 20000, "f32", seed=8, sigma=0.5)
    tau = 0.3 if div_kind == 1 else 0.5
    run_stage_both(psd, oracle, zs, zl, tok, tau, div_kind=div_kind, variant=psd.KERNEL_CLUSTER)
    zs, zl, tok = wl.make_stage_inputs(4, 4, 20000, "bf16", seed=8, sigma=0.5)
    zs[1, 1, 50:60] = -float("inf")             # KL(large || small) is +inf where small has no mass
    run_stage_both(psd, oracle, zs, zl, tok, tau, div_kind=div_kind, variant=psd.KERNEL_CLUSTER)


def test_cluster_occupancy_query(psd):
    cs, n = psd.cluster_occupancy(64, 16, 128256, psd.BF16)     # many rows: pairs of CTAs fill every SM
    assert cs == 2 and n >= 64
    cs, n = psd.cluster_occupancy(256, 8, 152064, psd.BF16)
    assert cs == 2 and n >= 64
    cs, n = psd.cluster_occupancy(4, 24, 128256, psd.BF16)      # 96 rows: three rounds of 33 clusters of 4 beat two of 74 pairs
    assert cs == 4 and n >= 16
    cs, n = psd.cluster_occupancy(256, 8, 152064, psd.F32)      # fp32: streamed twice on the smallest clusters whose rows in flight fit L2
    assert cs in (3, 4) and n >= 30
    cs, n = psd.cluster_occupancy(1, 4, 32000, psd.F32)
    assert cs >= 2 and n >= 1
    assert psd.cluster_occupancy(4, 4, 1001, psd.F32) == (0, 0)


# -------------------------------------------------------------------------------------------------- wrapper
def run_pyramid_both(psd, oracle, zd, zq, zt, tok, tau_q, tau_t, mode=0, seed=0, offset=0):
    dev = torch.device("cuda:0")
    out = psd.verify(zd.to(dev), zq.to(dev), zt.to(dev), tok.to(dev), tau_q, tau_t, mode, seed, offset)
    torch.cuda.synchronize()
    assert psd.last_status() == 0
    gpu = gpu_stage_to_numpy(out)
    zd_h, zq_h, zt_h = host_bits(zd), host_bits(zq), host_bits(zt)
    orc = oracle.verify(zd_h, zq_h, zt_h, tok.numpy(), np.float32(tau_q), np.float32(tau_t), mode, seed, offset,
                        n_threads=8)
    return gpu, orc, (zd_h, zq_h, zt_h)


def check_pyramid(oracle, gpu, orc, hosts, dtype, mode, tau_q, tau_t, seed, offset, tok, seq_ids=None):
    """Stage 1 against the oracle; when stage 1 agrees for a sequence, stage 2 must agree as well."""
    zd_h, zq_h, zt_h = hosts
    B, K_d = tok.shape
    K_q = zt_h.shape[1]
    s1g = dict(accept_len=gpu["accept_len_q"], next_token=gpu["next_token_q"])
    o1 = oracle.verify_stage(zd_h, zq_h, tok, np.float32(tau_q), mode, seed, offset, n_threads=8, seq_ids=seq_ids)
    assert np.array_equal(o1["accept_len"], orc["accept_len_q"])
    rep1 = compare_stage(oracle, s1g, o1, zd_h, zq_h, dtype=dtype, mode=mode, tau=float(np.float32(tau_q)), seed=seed,
                         offset=offset, seq_ids=seq_ids, check_rows=False)
    same = (gpu["accept_len_q"] == orc["accept_len_q"]) & (gpu["next_token_q"] == orc["next_token_q"])
    idx = np.nonzero(same)[0]
    rep2 = dict(tie_div=0, tie_coin=0, tie_cdf=0)
    if len(idx):
        zq2 = np.ascontiguousarray(zq_h[idx][:, :K_q])
        ids = idx if seq_ids is None else np.asarray(seq_ids)[idx]
        o2 = oracle.verify_stage(zq2, zt_h[idx], orc["window"][idx], np.float32(tau_t), mode, seed, offset + 1,
                                 n_valid=orc["n_window"][idx], n_threads=8, seq_ids=ids)
        assert np.array_equal(o2["accept_len"], orc["accept_len"][idx])
        s2g = dict(accept_len=gpu["accept_len"][idx], next_token=gpu["next_token"][idx])
        rep2 = compare_stage(oracle, s2g, o2, zq2, zt_h[idx], dtype=dtype, mode=mode, tau=float(np.float32(tau_t)),
                             seed=seed, offset=offset + 1, n_valid=orc["n_window"][idx], seq_ids=ids,
                             check_rows=False)
    ties = sum(rep1[k] + rep2[k] for k in ("tie_div", "tie_coin", "tie_cdf"))
    return ties, len(idx)


@pytest.mark.parametrize("mode", [0, 1])
def test_pyramid_reduced_cfg2(psd, oracle, wl, mode):
    """workload configuration 2 (single stream, V=128256 bf16, K_d=8, K_q=4), a few rounds."""
    ties = 0
    for rnd in range(3):
        zd, zq, zt, tok = wl.workload_inputs(2, rnd)
        gpu, orc, hosts = run_pyramid_both(psd, oracle, zd, zq, zt, tok, 0.4, 0.2, mode, 0, 2 * rnd)
        t, _ = check_pyramid(oracle, gpu, orc, hosts, "bf16", mode, 0.4, 0.2, 0, 2 * rnd, tok.numpy())
        ties += t
    assert ties <= 1


def test_pyramid_reduced_cfg3(psd, oracle, wl):
    """workload configuration 3 recipe at B=6 (V=128256 bf16, K_d=16, K_q=8, per-sequence boost U[4,12])."""
    zd, zq, zt, tok = wl.workload_inputs(3, 0, B=6)
    ties = 0
    for tau_q, tau_t in ((0.4, 0.2), (0.69, 0.5)):
        gpu, orc, hosts = run_pyramid_both(psd, oracle, zd, zq, zt, tok, tau_q, tau_t, 0, 0, 0)
        t, n = check_pyramid(oracle, gpu, orc, hosts, "bf16", 0, tau_q, tau_t, 0, 0, tok.numpy())
        ties += t
        assert n >= 5
    assert ties <= 1


def test_pyramid_small_vocab_all_paths(psd, oracle, wl):
    """Small V so that windows of every length (cut, short, full) occur; fp32; every mode."""
    zd, zq, zt, tok = wl.make_pyramid_inputs(24, 6, 4, 777, "f32", seed=21, sigma_q=0.3, sigma_d=0.5)
    for mode in (0, 1, 2, 3):
        gpu, orc, hosts = run_pyramid_both(psd, oracle, zd, zq, zt, tok, 0.03, 0.02, mode, 5, 10)
        ties, n = check_pyramid(oracle, gpu, orc, hosts, "f32", mode, 0.03, 0.02, 5, 10, tok.numpy())
        assert ties <= 2 and n >= 22
        lens = set(orc["n_window"].tolist())
        assert len(lens) >= 2


@pytest.mark.parametrize("K", [4, 8, 16, 32])
def test_cfg4_sweep_cells(psd, oracle, wl, K):
    """workload configuration 4 recipe (V=152064 bf16, qualifier noise 0.5, draft noise 2.0, boost 8) at B=2: every
    (K, tau) cell of the sweep, as the stage-1 pairing, the stage-2 pairing and the two-stage wrapper."""
    w = wl.CONFIGS[4]
    zd, zq, zt, tok = wl.make_pyramid_inputs(2, K, K, w.V, "bf16", seed=4000 + K, boost=w.boost, sigma_q=w.sigma_q,
                                             sigma_d=w.sigma_d)
    ties = 0
    for tau in wl.CFG4_TAU:
        _, o1, r1 = run_stage_both(psd, oracle, zd, zq, tok, tau, seed=0, offset=K)          # draft -> qualifier
        _, o2, r2 = run_stage_both(psd, oracle, zq, zt, tok, tau, seed=0, offset=K + 1)      # qualifier -> target
        ties += sum(r[k] for r in (r1, r2) for k in ("tie_div", "tie_cdf"))
        if tau >= 1.0:
            assert np.all(o1["accept_len"] == K) and np.all(o2["accept_len"] == K)   # tau >= max JS: all accepted
        Kq = max(K // 2, 1)
        gpu, orc, hosts = run_pyramid_both(psd, oracle, zd, zq, zt[:, :Kq].contiguous(), tok, tau, tau, 0, 0, 2 * K)
        t, _ = check_pyramid(oracle, gpu, orc, hosts, "bf16", 0, tau, tau, 0, 2 * K, tok.numpy())
        ties += t
    assert ties <= 2


def test_cfg4_fp32_k8(psd, oracle, wl):
    """Config 4's fp32 run at K=8 (B=2): the 1e-5 tolerance class on the large vocabulary."""
    w = wl.CONFIGS[4]
    zd, zq, zt, tok = wl.make_pyramid_inputs(2, 8, 8, w.V, "f32", seed=4999, boost=w.boost, sigma_q=w.sigma_q, sigma_d=w.sigma_d)
    for tau in (0.05, 0.5):
        _, _, rep = run_stage_both(psd, oracle, zq, zt, tok, tau, seed=0, offset=3)
        assert rep["max_err_div"] < 1e-5 and rep["max_err_prob"] < 1e-5
        _, _, rep = run_stage_both(psd, oracle, zd, zq, tok, tau, mode=1, seed=0, offset=4)
        assert rep["max_err_div"] < 1e-5


@pytest.mark.parametrize("B,K_d,K_q,V,dtype", [(9, 8, 4, 8192, "bf16"), (2, 8, 4, 65536, "bf16"), (3, 16, 8, 128256, "bf16"),
                                              (5, 5, 2, 32000, "f32")])
def test_two_stage_policies_give_the_same_results(psd, wl, B, K_d, K_q, V, dtype):
    """Few rows make the library widen its clusters; the stage-by-stage schedule sees fewer rows per launch than
    the single-launch one, and must still cut every row the same way."""
    dev = torch.device("cuda:0")
    zd, zq, zt, tok = [t.to(dev) for t in wl.make_pyramid_inputs(B, K_d, K_q, V, dtype, seed=23, sigma_q=0.6, sigma_d=1.2)]
    try:
        psd.set_two_stage_policy(psd.TWO_STAGE_FUSED)
        a = psd.verify(zd, zq, zt, tok, 0.3, 0.15, 2, 3, 4)
        torch.cuda.synchronize()
        psd.set_two_stage_policy(psd.TWO_STAGE_SEPARATE)
        b = psd.verify(zd, zq, zt, tok, 0.3, 0.15, 2, 3, 4)
        torch.cuda.synchronize()
    finally:
        psd.set_two_stage_policy(psd.TWO_STAGE_DEFAULT)
    for k in a:
        assert torch.equal(a[k], b[k]), k
    if B >= 9:
        assert 0 < int(a["accept_len_q"].sum()) < B * K_d


def test_two_stage_auto_policy_follows_the_window_lengths(psd, wl):
    """PSD_TWO_STAGE_AUTO: the first call of a shape takes the statistics of both stages in one launch; once stage 1
    has reported short windows the next call runs stage by stage (two statistics launches), and goes back when the
    windows are full again. The results are those of the fixed schedules, bit for bit."""
    dev = torch.device("cuda:0")
    B, K_d, K_q, V = 48, 16, 8, 8192            # 1152 rows
    zd, zq, zt, tok = [t.to(dev) for t in wl.make_pyramid_inputs(B, K_d, K_q, V, "bf16", seed=41, sigma_q=0.6, sigma_d=2.5)]
    psd.set_two_stage_policy(psd.TWO_STAGE_FUSED)
    ref_low = psd.verify(zd, zq, zt, tok, 0.02, 0.02, 0, 5, 6)      # tight threshold: short windows
    ref_full = psd.verify(zd, zq, zt, tok, 1.0, 1.0, 0, 5, 8)       # tau > ln 2: every window full
    torch.cuda.synchronize()
    psd.set_two_stage_policy(psd.TWO_STAGE_DEFAULT)
    assert float(ref_low["accept_len_q"].float().mean()) < 3 and int(ref_full["accept_len"].min()) == K_q
    try:
        psd.set_two_stage_policy(psd.TWO_STAGE_AUTO)
        launches = []
        # the lengths are sampled on every fourth call while the schedule is stage by stage: four calls with full
        # windows may pass before the library notices
        calls = [(0.02, 6, ref_low)] * 2 + [(1.0, 8, ref_full)] * 6
        for tau, offset, ref in calls:
            psd.kernel_timing_begin()
            out = psd.verify(zd, zq, zt, tok, tau, tau, 0, 5, offset)
            torch.cuda.synchronize()
            launches.append(psd.kernel_timing_end()[1])   # statistics launches of the call
            for k in ref:
                assert torch.equal(ref[k], out[k]), k
        assert launches[:2] == [1, 2] and launches[-1] == 1 and launches[2:] == sorted(launches[2:], reverse=True), launches
    finally:
        psd.set_two_stage_policy(psd.TWO_STAGE_DEFAULT)
    assert psd.last_status() == 0


def test_host_entry_point_equals_device_entry_point(psd, wl):
    dev = torch.device("cuda:0")
    zd, zq, zt, tok = wl.make_pyramid_inputs(5, 8, 4, 9000, "bf16", seed=22)
    a = psd.verify(zd.to(dev), zq.to(dev), zt.to(dev), tok.to(dev), 0.4, 0.2, 0, 3, 4)
    torch.cuda.synchronize()
    b = psd.verify_host(zd.pin_memory(), zq.pin_memory(), zt.pin_memory(), tok.pin_memory(), 0.4, 0.2, 0, 3, 4)
    for k in a:
        assert torch.equal(a[k].cpu(), b[k]), k


def test_full_size_bench_config_sampled(psd, oracle, wl):
    """The bench workload (config 3 at full size, B=64) in the launch configuration bench.py times;
    the oracle checks a sample of sequences one by one."""
    dev = torch.device("cuda:0")
    w = wl.CONFIGS[3]
    zd, zq, zt, tok = wl.workload_inputs(3, 1, device=dev)
    psd.set_stream()
    out = psd.verify(zd, zq, zt, tok, w.tau_q, w.tau_t, 0, 0, 2)
    torch.cuda.synchronize()
    assert psd.last_status() == 0
    pick = np.array([0, 13, 37, 63])
    gpu = {k: v.cpu().numpy()[pick] for k, v in out.items()}
    hosts = tuple(host_bits(t[pick]) for t in (zd, zq, zt))
    tok_h = tok.cpu().numpy()[pick]
    orc = oracle.verify(*hosts, tok_h, np.float32(w.tau_q), np.float32(w.tau_t), 0, 0, 2, n_threads=8, seq_ids=pick)
    ties, n = check_pyramid(oracle, gpu, orc, hosts, "bf16", 0, w.tau_q, w.tau_t, 0, 2, tok_h, seq_ids=pick)
    assert ties <= 1 and n >= 3
    # properties that hold for every sequence at any size
    al_q, nt_q = out["accept_len_q"].cpu().numpy(), out["next_token_q"].cpu().numpy()
    al, nt = out["accept_len"].cpu().numpy(), out["next_token"].cpu().numpy()
    assert np.all((0 <= al_q) & (al_q <= w.K_d)) and np.all((nt_q >= 0) == (al_q < w.K_d))
    n2 = np.minimum(w.K_q, al_q + (nt_q >= 0))
    assert np.all(al <= n2) and np.all((nt >= 0) == (al < n2)) and np.all(nt < w.V)
