"""GPU parity of the extended two-stage call (pyramidsd_verify_ex): per-stage acceptance modes (the assisted
variant of Sec. 3.4), per-row outputs, the sequence base that lets a shard reproduce the unsharded call, the
row-triple schedule, the workload-4 launch configuration at full size, per-stream scratch, and the path by which a
bounded device wait reports that it gave up."""
import threading

import numpy as np
import pytest
import torch

from parity_utils import TOL, compare_stage, gpu_stage_to_numpy, host_bits

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


def bits(t):
    return t.view(torch.int32) if t.dtype == torch.float32 else t


def check_pyramid_ex(oracle, gpu, hosts, tok, dtype, mode_q, mode_t, tau_q, tau_t, seed, offset, seq_ids=None):
    """Both stages against the oracle, element by element where the library reports rows: stage 1 always; stage 2
    for the sequences whose stage-1 integers agree (the window is then the oracle's)."""
    zd_h, zq_h, zt_h = hosts
    K_q = zt_h.shape[1]
    orc = oracle.verify(zd_h, zq_h, zt_h, tok, np.float32(tau_q), np.float32(tau_t), mode_q, seed, offset, n_threads=8,
                        seq_ids=seq_ids, mode_t=mode_t)
    o1 = oracle.verify_stage(zd_h, zq_h, tok, np.float32(tau_q), mode_q, seed, offset, n_threads=8, seq_ids=seq_ids)
    g1 = dict(accept_len=gpu["accept_len_q"], next_token=gpu["next_token_q"], div=gpu["div_q"], resid_mass=gpu["resid_q"])
    tol = TOL[dtype]["val"]
    fin = np.isfinite(o1["div"])
    assert np.abs(g1["div"][fin] - o1["div"][fin]).max() <= tol
    assert np.abs(g1["resid_mass"][fin] - o1["resid_mass"][fin]).max() <= tol
    rep1 = compare_stage(oracle, g1, o1, zd_h, zq_h, dtype=dtype, mode=mode_q, tau=float(np.float32(tau_q)), seed=seed,
                         offset=offset, seq_ids=seq_ids, check_rows=False)
    same = (gpu["accept_len_q"] == orc["accept_len_q"]) & (gpu["next_token_q"] == orc["next_token_q"])
    idx = np.nonzero(same)[0]
    assert np.array_equal(gpu["window"][idx], orc["window"][idx]) and np.array_equal(gpu["n_window"][idx], orc["n_window"][idx])
    rep2 = dict(tie_div=0, tie_coin=0, tie_cdf=0)
    if len(idx):
        zq2 = np.ascontiguousarray(zq_h[idx][:, :K_q])
        ids = idx if seq_ids is None else np.asarray(seq_ids)[idx]
        o2 = oracle.verify_stage(zq2, zt_h[idx], orc["window"][idx], np.float32(tau_t), mode_t, seed, offset + 1,
                                 n_valid=orc["n_window"][idx], n_threads=8, seq_ids=ids)
        assert np.array_equal(o2["accept_len"], orc["accept_len"][idx])
        valid = np.arange(K_q)[None, :] < orc["n_window"][idx][:, None]
        ok = valid & np.isfinite(o2["div"])
        assert np.abs(gpu["div_t"][idx][ok] - o2["div"][ok]).max() <= tol
        assert np.abs(gpu["resid_t"][idx][ok] - o2["resid_mass"][ok]).max() <= tol
        assert np.all(gpu["div_t"][idx][~valid] == 0)
        g2 = dict(accept_len=gpu["accept_len"][idx], next_token=gpu["next_token"][idx])
        rep2 = compare_stage(oracle, g2, o2, zq2, zt_h[idx], dtype=dtype, mode=mode_t, tau=float(np.float32(tau_t)),
                             seed=seed, offset=offset + 1, n_valid=orc["n_window"][idx], seq_ids=ids, check_rows=False)
    ties = sum(rep1[k] + rep2[k] for k in ("tie_div", "tie_coin", "tie_cdf"))
    return ties, len(idx), orc


@pytest.mark.parametrize("dtype,V", [("f32", 777), ("bf16", 32768)])
def test_assisted_qualifier_stage_with_fuzzy_target_stage(psd, oracle, wl, dtype, V):
    """PSD_A (Sec. 3.4): stage 1 accepts by the coin flip and falls back to a draw from the qualifier itself, stage 2
    keeps its threshold; also every other pairing of modes once, and rows, window and lengths element by element."""
    dev = torch.device("cuda:0")
    B, K_d, K_q = 20, 6, 4
    zd, zq, zt, tok = wl.make_pyramid_inputs(B, K_d, K_q, V, dtype, seed=71, sigma_q=0.3, sigma_d=0.6)
    hosts = tuple(host_bits(t) for t in (zd, zq, zt))
    dd = [t.to(dev) for t in (zd, zq, zt, tok)]
    total = 0
    for mode_q, mode_t, tau_q, tau_t in ((psd.ASSISTED, psd.FUZZY, 0.0, 0.03), (psd.FUZZY, psd.STRICT, 0.05, 0.0),
                                         (psd.STRICT, psd.FUZZY_SD_FALLBACK, 0.0, 0.02), (psd.FUZZY, psd.FUZZY, 0.05, 0.03)):
        out = psd.verify_ex(*dd, tau_q, tau_t, mode_q, mode_t, 9, 30)
        torch.cuda.synchronize()
        assert psd.last_status() == 0
        gpu = gpu_stage_to_numpy(out)
        ties, n, orc = check_pyramid_ex(oracle, gpu, hosts, tok.numpy(), dtype, mode_q, mode_t, tau_q, tau_t, 9, 30)
        total += ties
        assert n >= B - 2
        assert 0 < orc["accept_len_q"].sum() < B * K_d and len(set(orc["n_window"].tolist())) >= 2
    assert total <= 3


def test_sequence_base_makes_shards_reproduce_the_whole_batch(psd, wl):
    """The whole batch in one call equals its shards in calls of their own -- every accept length, token, window --
    when each shard passes the index of its first sequence: the coin flips and draws of a row are those of its index in the whole batch. Stage
    and pyramid, coin-flip and threshold modes, the bonus draw, ragged shards of two and three ranks."""
    dev = torch.device("cuda:0")
    B, K_d, K_q, V = 11, 6, 3, 8192
    zd, zq, zt, tok = [t.to(dev) for t in wl.make_pyramid_inputs(B, K_d, K_q + 1, V, "bf16", seed=81, sigma_q=0.4, sigma_d=0.8)]
    zt_plain = zt[:, :K_q].contiguous()
    for world in (2, 3):
        for mode in (psd.STRICT, psd.FUZZY, psd.ASSISTED):
            full_s = psd.verify_stage_ex(zd, zq, tok, 0.05, mode, 4, 12)
            full_p = psd.verify_ex(zd, zq, zt_plain, tok, 0.05, 0.03, mode, None, 4, 12)
            full_b = psd.verify_ex(zd, zq, zt, tok, 0.6, 0.6, psd.FUZZY, mode, 4, 12, target_has_bonus_row=True)
            torch.cuda.synchronize()
            assert 0 < int(full_s["accept_len"].sum()) < B * K_d
            assert int((full_b["accept_len"] == full_b["n_window"]).sum()) > 0 or mode != psd.FUZZY   # bonus draws happen
            for rank in range(world):
                lo, hi, base = wl.shard_call(B, rank, world)
                sl = slice(lo, hi)
                part_s = psd.verify_stage_ex(zd[sl].contiguous(), zq[sl].contiguous(), tok[sl].contiguous(), 0.05, mode, 4, 12,
                                             seq_index_base=base)
                part_p = psd.verify_ex(zd[sl].contiguous(), zq[sl].contiguous(), zt_plain[sl].contiguous(), tok[sl].contiguous(),
                                       0.05, 0.03, mode, None, 4, 12, seq_index_base=base)
                part_b = psd.verify_ex(zd[sl].contiguous(), zq[sl].contiguous(), zt[sl].contiguous(), tok[sl].contiguous(),
                                       0.6, 0.6, psd.FUZZY, mode, 4, 12, target_has_bonus_row=True, seq_index_base=base)
                torch.cuda.synchronize()
                for full, part in ((full_s, part_s), (full_p, part_p), (full_b, part_b)):
                    for k, v in part.items():
                        if not torch.is_tensor(v):
                            continue
                        if v.dtype == torch.int32:
                            assert torch.equal(v, full[k][sl]), (world, mode, rank, k)
                        else:   # a smaller call may cut its rows over another number of CTAs: last-bit differences
                            assert torch.allclose(v, full[k][sl], rtol=0, atol=5e-6, equal_nan=True), (world, mode, rank, k)
    # without the base a shard draws other numbers: the test above is not vacuous
    lo, hi, base = wl.shard_call(B, 1, 2)
    wrong = psd.verify_stage_ex(zd[lo:hi].contiguous(), zq[lo:hi].contiguous(), tok[lo:hi].contiguous(), 0.05, psd.STRICT, 4, 12)
    right = psd.verify_stage_ex(zd, zq, tok, 0.05, psd.STRICT, 4, 12)
    torch.cuda.synchronize()
    assert not (torch.equal(wrong["accept_len"], right["accept_len"][lo:hi]) and
                torch.equal(wrong["next_token"], right["next_token"][lo:hi]))
    assert psd.last_status() == 0


@pytest.mark.parametrize("B,K_d,K_q,V,dtype", [(24, 16, 8, 128256, "bf16"), (40, 8, 4, 152064, "bf16"), (30, 6, 6, 152064, "f32"),
                                              (3, 8, 4, 32768, "bf16")])
def test_every_schedule_returns_the_same_bits(psd, wl, B, K_d, K_q, V, dtype):
    """Two launches over row pairs, two launches over row triples (where the statistics kernel streams its rows
    twice: the first three shapes), stage by stage, and the per-call choice: the same integers, divergences and
    residual masses, bit for bit, in a threshold mode and in a coin-flip mode."""
    dev = torch.device("cuda:0")
    zd, zq, zt, tok = [t.to(dev) for t in wl.make_pyramid_inputs(B, K_d, K_q, V, dtype, seed=91, boost=(4.0, 12.0),
                                                                 sigma_q=0.6, sigma_d=1.2)]
    probe = psd.verify_ex(zd, zq, zt, tok, 1.0, 1.0, psd.FUZZY, None, 3, 4, schedule=psd.TWO_STAGE_FUSED)
    tau_q = float(probe["div_q"].quantile(0.85))     # thresholds that leave windows of every length
    tau_t = float(probe["div_t"].quantile(0.7))
    for mode in (psd.FUZZY, psd.FUZZY_SD_FALLBACK):
        ref = None
        for sched in (psd.TWO_STAGE_FUSED, psd.TWO_STAGE_FUSED_ROWS, psd.TWO_STAGE_SEPARATE, psd.TWO_STAGE_AUTO, psd.TWO_STAGE_AUTO):
            out = psd.verify_ex(zd, zq, zt, tok, tau_q, tau_t, mode, None, 3, 4, schedule=sched)
            torch.cuda.synchronize()
            assert psd.last_status() == 0
            if ref is None:
                ref = out
                assert 0 < int(out["accept_len_q"].sum()) < B * K_d
                continue
            valid = torch.arange(K_q, device=dev)[None, :] < out["n_window"][:, None]
            for k, v in out.items():
                if not torch.is_tensor(v):
                    continue
                if k in ("div_t", "resid_t"):   # rows beyond a window are not scored by the stage-by-stage schedule
                    assert torch.equal(bits(v)[valid], bits(ref[k])[valid]), (sched, k)
                else:
                    assert torch.equal(bits(v), bits(ref[k])), (sched, k)


def test_row_triples_against_the_oracle(psd, oracle, wl):
    """The row-triple schedule element by element against the oracle on the workload-3 recipe at B=12 (more work items
    than clusters would need B >= 5: 192 items over 74 pairs of CTAs), with masked and poisoned rows among them."""
    dev = torch.device("cuda:0")
    B, K_d, K_q, V = 12, 16, 8, 128256
    zd, zq, zt, tok = wl.workload_inputs(3, 7, B=B)
    zq[1, 2, 1000:90000] = -float("inf")      # masked vocabulary in the row both stages share
    zt[2, 1, 77] = float("nan")               # a poisoned target row: stage 2 rejects there
    zd[3, 0] = zq[3, 0]                       # bitwise identical stage-1 pair
    zt[4, 3] = zq[4, 3]                       # bitwise identical stage-2 pair
    zq[5, 4, 120000] = 300.0                  # far above the row's first vectors: the optimistic sums overflow
    hosts = tuple(host_bits(t) for t in (zd, zq, zt))
    assert psd.cluster_occupancy(B, K_d + K_q, V, psd.BF16)[0] == 2      # pairs of CTAs: streamed twice
    out = psd.verify_ex(zd.to(dev), zq.to(dev), zt.to(dev), tok.to(dev), 0.4, 0.2, psd.FUZZY, None, 0, 14,
                        schedule=psd.TWO_STAGE_FUSED_ROWS)
    torch.cuda.synchronize()
    assert psd.last_status() == 0
    gpu = gpu_stage_to_numpy(out)
    ties, n, orc = check_pyramid_ex(oracle, gpu, hosts, tok.numpy(), "bf16", 0, 0, 0.4, 0.2, 0, 14)
    assert ties <= 1 and n >= B - 1
    assert gpu["div_q"][3, 0] == 0.0 and gpu["resid_q"][3, 0] == 0.0
    if gpu["n_window"][4] > 3:
        assert gpu["div_t"][4, 3] == 0.0
    if gpu["n_window"][2] > 1 and gpu["accept_len"][2] >= 1:
        assert gpu["accept_len"][2] == 1 and gpu["next_token"][2] == -2


def test_full_size_cfg4_sampled(psd, oracle, wl):
    """Workload 4 at the size and in the launch configurations bench.py times it in -- B=256, V=152064, K_d=8, K_q=4,
    tau=0.2; bf16 under every schedule, fp32 stage by stage -- with the oracle on sampled sequences (their Philox
    rows are those of the full batch), rows compared element by element."""
    dev = torch.device("cuda:0")
    w = wl.CONFIGS[4]
    pick = np.array([0, 101, 180, 255])
    for dtype, schedules in (("bf16", (psd.TWO_STAGE_FUSED, psd.TWO_STAGE_SEPARATE, psd.TWO_STAGE_DEFAULT, psd.TWO_STAGE_FUSED_ROWS)),
                             ("f32", (psd.TWO_STAGE_SEPARATE,))):
        zd, zq, zt, tok = wl.make_pyramid_inputs(w.B, w.K_d, w.K_q, w.V, dtype, 4000, w.boost, w.sigma_q, w.sigma_d, device=dev)
        hosts = tuple(host_bits(t[pick]) for t in (zd, zq, zt))
        tok_h = tok.cpu().numpy()[pick]
        first = None
        for sched in schedules:
            out = psd.verify_ex(zd, zq, zt, tok, w.tau_q, w.tau_t, psd.FUZZY, None, 0, 6, schedule=sched)
            torch.cuda.synchronize()
            assert psd.last_status() == 0
            al_q, nt_q = out["accept_len_q"].cpu().numpy(), out["next_token_q"].cpu().numpy()
            al, nt = out["accept_len"].cpu().numpy(), out["next_token"].cpu().numpy()
            n2 = np.minimum(w.K_q, al_q + (nt_q >= 0))
            assert np.all((0 <= al_q) & (al_q <= w.K_d)) and np.all((nt_q >= 0) == (al_q < w.K_d))
            assert np.array_equal(out["n_window"].cpu().numpy(), n2)
            assert np.all(al <= n2) and np.all((nt >= 0) == (al < n2)) and np.all(nt < w.V)
            if first is None:
                first = out
                gpu = {k: v.cpu().numpy()[pick] for k, v in out.items() if torch.is_tensor(v)}
                ties, n, _ = check_pyramid_ex(oracle, gpu, hosts, tok_h, dtype, 0, 0, w.tau_q, w.tau_t, 0, 6, seq_ids=pick)
                assert ties <= 1 and n >= 3
            else:
                for k in ("accept_len_q", "next_token_q", "accept_len", "next_token", "div_q", "resid_q", "window", "n_window"):
                    assert torch.equal(bits(out[k]), bits(first[k])), (dtype, sched, k)
        del zd, zq, zt, tok, first, out
        torch.cuda.empty_cache()


def test_bounded_wait_that_runs_out_is_reported_and_leaves_the_library_usable(psd, wl):
    """A kernel whose only wait can never be satisfied gives up after its poll limit, ends normally, and the status
    call says so once; the next verification on the same stream is clean and correct."""
    dev = torch.device("cuda:0")
    zs, zl, tok = [t.to(dev) for t in wl.make_stage_inputs(4, 4, 8192, "bf16", seed=95, sigma=0.5)]
    ref = psd.verify_stage_ex(zs, zl, tok, 0.05, psd.STRICT, 1, 2)
    torch.cuda.synchronize()
    assert psd.last_status() == psd.OK
    assert psd.selftest_wait_timeout() == psd.OK
    assert psd.last_status() == psd.ERR_TIMEOUT
    assert psd.last_status() == psd.OK                # reading the status clears it
    out = psd.verify_stage_ex(zs, zl, tok, 0.05, psd.STRICT, 1, 2)
    torch.cuda.synchronize()
    assert psd.last_status() == psd.OK
    for k, v in ref.items():
        if torch.is_tensor(v):
            assert torch.equal(bits(v), bits(out[k])), k
    # the status belongs to the stream: a timeout recorded on one stream does not show on another
    side = torch.cuda.Stream()
    assert psd.selftest_wait_timeout(side) == psd.OK
    side.synchronize()
    psd.verify_stage_ex(zs, zl, tok, 0.05, psd.STRICT, 1, 2)
    assert psd.last_status() == psd.OK
    assert psd.selftest_wait_timeout(side) == psd.OK  # makes `side` the stream of this thread's most recent call
    assert psd.last_status() == psd.ERR_TIMEOUT


def test_streams_and_host_threads_do_not_share_scratch(psd, wl):
    """Calls of different sizes issued from two host threads on two streams, interleaved on the device: every result
    equals the one the same call gives alone. Each stream has scratch of its own, and a call can bring its own."""
    dev = torch.device("cuda:0")
    cases = []
    for i, (B, K_d, K_q, V) in enumerate(((48, 8, 4, 32768), (6, 16, 8, 65536))):
        t = [x.to(dev) for x in wl.make_pyramid_inputs(B, K_d, K_q, V, "bf16", seed=97 + i, sigma_q=0.5, sigma_d=1.0)]
        ref = psd.verify_ex(*t, 0.3, 0.15, psd.FUZZY_SD_FALLBACK, None, 2, 8)
        torch.cuda.synchronize()
        cases.append((t, ref))
    errors = []

    def worker(idx):
        try:
            torch.cuda.set_device(0)
            stream = torch.cuda.Stream()
            t, ref = cases[idx]
            with torch.cuda.stream(stream):
                for it in range(40):
                    out = psd.verify_ex(*t, 0.3, 0.15, psd.FUZZY_SD_FALLBACK, None, 2, 8, stream=stream)
                    if it % 8 == 7:
                        stream.synchronize()
                        for k, v in ref.items():
                            if torch.is_tensor(v) and not torch.equal(bits(v), bits(out[k])):
                                errors.append((idx, it, k))
                stream.synchronize()
                if psd.last_status() != psd.OK:
                    errors.append((idx, "status"))
        except Exception as e:   # noqa: BLE001
            errors.append((idx, repr(e)))

    threads = [threading.Thread(target=worker, args=(i,)) for i in range(2)]
    for th in threads:
        th.start()
    for th in threads:
        th.join()
    assert not errors, errors[:5]
    # a caller workspace: no library-owned statistics buffer is involved
    t, ref = cases[0]
    B, K_d, V = t[0].shape
    need = psd.pyramid_workspace_bytes(B, K_d, t[2].shape[1], V, psd.BF16)
    ws = torch.empty(need, dtype=torch.uint8, device=dev)
    out = psd.verify_ex(*t, 0.3, 0.15, psd.FUZZY_SD_FALLBACK, None, 2, 8, workspace=ws)
    torch.cuda.synchronize()
    for k, v in ref.items():
        if torch.is_tensor(v):
            assert torch.equal(bits(v), bits(out[k])), k
    # more streams than the library keeps scratch for: the call says so, releasing a stream makes room again
    streams = [torch.cuda.Stream() for _ in range(20)]
    codes = [psd.verify_ex(*t, 0.3, 0.15, stream=st, raise_on_error=False, want_rows=False, want_window=False)["status"] for st in streams]
    torch.cuda.synchronize()
    assert codes[0] == psd.OK and psd.ERR_WORKSPACE in codes and set(codes) <= {psd.OK, psd.ERR_WORKSPACE}
    refused = streams[codes.index(psd.ERR_WORKSPACE)]
    with_ws = psd.verify_ex(*t, 0.3, 0.15, psd.FUZZY_SD_FALLBACK, None, 2, 8, stream=refused, workspace=ws)   # needs no library buffer
    refused.synchronize()
    assert torch.equal(with_ws["accept_len"], ref["accept_len"]) and psd.last_status() == psd.OK
    for st, code in zip(streams, codes):
        if code == psd.OK:
            psd.release_stream(st)
    out = psd.verify_ex(*t, 0.3, 0.15, psd.FUZZY_SD_FALLBACK, None, 2, 8, stream=refused)
    refused.synchronize()
    assert torch.equal(out["accept_len"], ref["accept_len"]) and torch.equal(out["next_token"], ref["next_token"])
    psd.release_stream(refused)
    small = torch.empty(need - 256, dtype=torch.uint8, device=dev)
    assert psd.verify_ex(*t, 0.3, 0.15, workspace=small, raise_on_error=False)["status"] == psd.ERR_WORKSPACE


def test_rejected_row_whose_residual_vanishes_in_single_precision_still_draws(psd, oracle, wl):
    """Two rows that differ only where both probabilities underflow (one side masks tokens the other gives a logit of
    -200): the residual mass is positive but below what single precision resolves. A rejection there draws from
    p_large, so next_token is a token (never -1) and both schedules of the pyramid agree. Against the oracle, which
    resolves a residual mass of 1e-90, the disagreements fall in the counted classes: |D - tau| < 1e-4 for the
    threshold decision at tau = 0, "residual below 1e-6" for the draw."""
    dev = torch.device("cuda:0")
    B, K, V = 3, 4, 4096
    zs, zl, tok = wl.make_stage_inputs(B, K, V, "f32", seed=99, sigma=0.0)
    zl[:, :, 100:140] = -200.0
    zs[:, :, 100:140] = -float("inf")
    out = psd.verify_stage_ex(zs.to(dev), zl.to(dev), tok.to(dev), -1.0)        # tau < 0: every row is rejected
    torch.cuda.synchronize()
    assert out["accept_len"].tolist() == [0] * B and bool((out["next_token"] >= 0).all())
    assert bool(((out["next_token"] < 100) | (out["next_token"] >= 140)).all())      # a token the large model can emit
    gpu = gpu_stage_to_numpy(psd.verify_stage_ex(zs.to(dev), zl.to(dev), tok.to(dev), 0.0))
    orc = oracle.verify_stage(host_bits(zs), host_bits(zl), tok.numpy(), np.float32(0.0), n_threads=4)
    assert np.all(orc["div"] > 0) and np.all(orc["div"] < 1e-30)
    rep = compare_stage(oracle, gpu, orc, host_bits(zs), host_bits(zl), dtype="f32", mode=0, tau=0.0, seed=0, offset=0)
    assert rep["tie_div"] == int((gpu["accept_len"] != orc["accept_len"]).sum()) and rep["tie_cdf"] == 0
    assert rep["tie_div"] + rep["tie_resid"] == B
    zt = zl[:, :2].clone()
    a = psd.verify_ex(zs.to(dev), zl.to(dev), zt.to(dev), tok.to(dev), -1.0, 0.5, schedule=psd.TWO_STAGE_FUSED)
    b = psd.verify_ex(zs.to(dev), zl.to(dev), zt.to(dev), tok.to(dev), -1.0, 0.5, schedule=psd.TWO_STAGE_SEPARATE)
    torch.cuda.synchronize()
    for k in ("accept_len_q", "next_token_q", "accept_len", "next_token", "n_window", "window"):
        assert torch.equal(a[k], b[k]), k
    assert a["n_window"].tolist() == [1] * B and int(a["accept_len"].max()) <= 1
    assert psd.last_status() == 0


def test_total_variation_through_every_schedule(psd, oracle, wl):
    """div_kind = total variation (three ex2 per index pair: pass B needs max(p, q) only) in the two-stage call: every
    schedule, row triples included, returns the same bits, and the per-row divergences are the oracle's."""
    dev = torch.device("cuda:0")
    B, K_d, K_q, V = 24, 6, 4, 32768
    zd, zq, zt, tok = wl.make_pyramid_inputs(B, K_d, K_q, V, "bf16", seed=45, sigma_q=0.3, sigma_d=0.6)
    dd = [t.to(dev) for t in (zd, zq, zt, tok)]
    probe = psd.verify_ex(*dd, 1e9, 1e9, div_kind=psd.DIV_TV)
    tau_q, tau_t = float(probe["div_q"].median()), float(probe["div_t"].median())
    outs = []
    for schedule in (psd.TWO_STAGE_FUSED, psd.TWO_STAGE_SEPARATE, psd.TWO_STAGE_FUSED_ROWS, psd.TWO_STAGE_AUTO):
        outs.append(psd.verify_ex(*dd, tau_q, tau_t, psd.FUZZY, psd.FUZZY, 5, 9, div_kind=psd.DIV_TV, schedule=schedule))
        torch.cuda.synchronize()
        assert psd.last_status() == 0
    for o in outs[1:]:
        for k in ("accept_len_q", "next_token_q", "accept_len", "next_token", "window", "n_window", "div_q", "resid_q"):
            assert torch.equal(bits(outs[0][k]), bits(o[k])), k
    gpu = gpu_stage_to_numpy(outs[0])
    o1 = oracle.verify_stage(host_bits(zd), host_bits(zq), tok.numpy(), np.float32(tau_q), 0, 5, 9, div_kind=1, n_threads=8)
    orc = oracle.verify(host_bits(zd), host_bits(zq), host_bits(zt), tok.numpy(), np.float32(tau_q), np.float32(tau_t), 0, 5, 9,
                        div_kind=1, n_threads=8)
    assert np.abs(gpu["div_q"] - o1["div"]).max() <= TOL["bf16"]["val"]
    assert np.abs(gpu["div_q"] - gpu["resid_q"]).max() == 0.0        # the total variation is the residual mass
    same = (gpu["accept_len_q"] == orc["accept_len_q"]) & (gpu["next_token_q"] == orc["next_token_q"])
    assert same.sum() >= B - 2 and np.array_equal(gpu["accept_len"][same], orc["accept_len"][same])
    assert 0 < orc["accept_len_q"].sum() < B * K_d
