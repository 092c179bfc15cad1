"""GPU tests of the two forms of the finalisation (accept scan, prefix, residual draw: Sec. 3.1, 3.2, 3.4). A large batch
that uses the library's own scratch is finalised in three launches (scan, tile totals, pick); the same call with a
caller workspace keeps the one-launch form, a cluster per sequence. Both must return the same bits -- checked here on
every acceptance mode, masked and flagged rows, ragged n_valid, a residual that vanishes in single precision, and the
two stages of a pyramid side by side -- and the three-launch form is compared with the oracle as well."""
import numpy as np
import pytest
import torch

from parity_utils import compare_stage, gpu_stage_to_numpy, host_bits
from test_gpu_pyramid_ex import check_pyramid_ex

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


def spoil(zs, zl, tok, V):
    """Rows of every special kind, in place: a NaN, a row with no finite entry, a token out of range, a one-sided mask
    and a pair whose residual vanishes in single precision."""
    zs[1, 0, 17] = float("nan")
    zl[2, 1, :] = -float("inf")
    tok[3, 0] = V
    zs[4, 1, 100:900] = -float("inf")
    zl[5, :, :] = zs[5, :, :]
    zl[5, :, 100:140] = -200.0
    zs[5, :, 100:140] = -float("inf")


@pytest.mark.parametrize("dtype,V", [("bf16", 20000), ("f32", 20004), ("bf16", 8191)])
def test_three_launches_equal_one_launch_single_stage(psd, wl, dtype, V):
    dev = torch.device("cuda:0")
    B, K = 100, 5
    zs, zl, tok = wl.make_stage_inputs(B, K, V, dtype, seed=500 + V, sigma=0.6)
    spoil(zs, zl, tok, V)
    n_valid = torch.as_tensor(np.random.default_rng(V).integers(0, K + 1, size=B), dtype=torch.int32)
    n_valid[:8] = K
    zs, zl, tok, n_valid = zs.to(dev), zl.to(dev), tok.to(dev), n_valid.to(dev)
    ws = torch.empty(psd.workspace_bytes(B, K, V, psd.dtype_code(zs)), dtype=torch.uint8, device=dev)
    drew = 0
    for mode in (psd.FUZZY, psd.STRICT, psd.FUZZY_SD_FALLBACK, psd.ASSISTED):
        for tau in (-1.0, 0.03):
            n0 = psd.launch_count()
            a = psd.verify_stage_ex(zs, zl, tok, tau, mode, 7, 3, n_valid=n_valid)
            n1 = psd.launch_count()
            b = psd.verify_stage_ex(zs, zl, tok, tau, mode, 7, 3, n_valid=n_valid, workspace=ws)
            n2 = psd.launch_count()
            torch.cuda.synchronize()
            assert psd.last_status() == 0
            assert (n1 - n0, n2 - n1) == (4, 2)    # statistics + scan, tiles, pick; statistics + one finalisation
            for k in a:
                if torch.is_tensor(a[k]):
                    x, y = a[k], b[k]
                    if x.dtype == torch.float32:
                        x, y = x.view(torch.int32), y.view(torch.int32)
                    assert torch.equal(x, y), (mode, tau, k)
            drew += int((a["next_token"] >= 0).sum())
            assert int(a["next_token"][1]) == -2 and int(a["accept_len"][1]) == 0     # the NaN row ends sequence 1
    assert drew > 2 * B


@pytest.mark.parametrize("mode_q", [0, 1, 3])    # threshold, coin flip, assisted (PSD_A of Sec. 3.4 with stage 2 fuzzy)
def test_three_launches_equal_one_launch_pyramid(psd, oracle, wl, mode_q):
    dev = torch.device("cuda:0")
    B, K_d, K_q, V = 60, 6, 4, 24576
    zd, zq, zt, tok = wl.make_pyramid_inputs(B, K_d, K_q, V, "bf16", seed=61, sigma_q=0.3, sigma_d=0.6)
    zq[2, 1, :] = -float("inf")
    zd[7, 0, 33] = float("nan")
    dd = [t.to(dev) for t in (zd, zq, zt, tok)]
    probe = psd.verify_ex(*dd, 1e9, 1e9)
    tau_q = float(probe["div_q"][torch.isfinite(probe["div_q"])].median())
    tau_t = float(probe["div_t"][torch.isfinite(probe["div_t"])].median())
    ws = torch.empty(psd.pyramid_workspace_bytes(B, K_d, K_q, V, psd.dtype_code(dd[0])), dtype=torch.uint8, device=dev)
    for schedule in (psd.TWO_STAGE_FUSED, psd.TWO_STAGE_FUSED_ROWS):
        n0 = psd.launch_count()
        a = psd.verify_ex(*dd, tau_q, tau_t, mode_q, psd.FUZZY, 5, 9, schedule=schedule)
        n1 = psd.launch_count()
        b = psd.verify_ex(*dd, tau_q, tau_t, mode_q, psd.FUZZY, 5, 9, schedule=schedule, workspace=ws)
        n2 = psd.launch_count()
        torch.cuda.synchronize()
        assert psd.last_status() == 0
        assert (n1 - n0, n2 - n1) == (4, 2)
        for k in a:
            if torch.is_tensor(a[k]):
                x, y = a[k], b[k]
                if x.dtype == torch.float32:
                    x, y = x.view(torch.int32), y.view(torch.int32)
                assert torch.equal(x, y), k
        assert 0 < int(a["accept_len_q"].sum()) < B * K_d and int((a["next_token"] >= 0).sum()) > 0
    # and against the oracle, without the two spoiled sequences' rows in the way of the helper's element-wise checks
    keep = [i for i in range(B) if i not in (2, 7)]
    sub = [t[keep].contiguous() for t in (zd, zq, zt, tok)]
    out = psd.verify_ex(*[t.to(dev) for t in sub], tau_q, tau_t, mode_q, psd.FUZZY, 5, 9)
    torch.cuda.synchronize()
    ties, n, orc = check_pyramid_ex(oracle, gpu_stage_to_numpy(out), tuple(host_bits(t) for t in sub[:3]), sub[3].numpy(),
                                    "bf16", mode_q, psd.FUZZY, tau_q, tau_t, 5, 9)
    assert ties <= 3 and n >= len(keep) - 2


@pytest.mark.parametrize("mode", [0, 1, 3])
def test_three_launch_form_against_oracle(psd, oracle, wl, mode):
    dev = torch.device("cuda:0")
    B, K, V = 96, 4, 12000
    zs, zl, tok = wl.make_stage_inputs(B, K, V, "f32", seed=77 + mode, sigma=0.6)
    spoil(zs, zl, tok, V)
    ties = 0
    for offset in range(2):
        n0 = psd.launch_count()
        out = psd.verify_stage_ex(zs.to(dev), zl.to(dev), tok.to(dev), 0.05, mode, 3, offset)
        torch.cuda.synchronize()
        assert psd.launch_count() - n0 == 4 and psd.last_status() == 0
        gpu = gpu_stage_to_numpy(out)
        orc = oracle.verify_stage(host_bits(zs), host_bits(zl), tok.numpy(), np.float32(0.05), mode, 3, offset, n_threads=8)
        rep = compare_stage(oracle, gpu, orc, host_bits(zs), host_bits(zl), dtype="f32", mode=mode,
                            tau=float(np.float32(0.05)), seed=3, offset=offset)
        ties += rep["tie_coin"] + rep["tie_cdf"] + rep["tie_div"]
        assert rep["tie_resid"] <= K      # sequence 5's rows, whose residual single precision cannot tell from zero
        assert 0 < orc["accept_len"].sum() < B * K
    assert ties <= 4


def test_three_launch_form_on_two_streams_from_two_threads(psd, wl):
    """The draw records and tile totals belong to the stream a call runs on: two host threads, each on a stream of its
    own, issue three-launch finalisations of different shapes back to back; every result equals the one the same call
    gives alone."""
    import threading
    dev = torch.device("cuda:0")
    cases = []
    t = [x.to(dev) for x in wl.make_pyramid_inputs(48, 8, 4, 32768, "bf16", seed=131, sigma_q=0.4, sigma_d=0.8)]
    probe = psd.verify_ex(*t, 1e9, 1e9)
    tau_q, tau_t = float(probe["div_q"].median()), float(probe["div_t"].median())
    call_a = lambda **kw: psd.verify_ex(*t, tau_q, tau_t, psd.FUZZY, psd.FUZZY, 2, 8, schedule=psd.TWO_STAGE_FUSED, **kw)
    s = [x.to(dev) for x in wl.make_stage_inputs(100, 5, 20000, "f32", seed=132, sigma=0.6)]
    call_b = lambda **kw: psd.verify_stage_ex(*s, 0.03, psd.STRICT, 4, 1, **kw)
    for call in (call_a, call_b):
        n0 = psd.launch_count()
        ref = call()
        torch.cuda.synchronize()
        assert psd.launch_count() - n0 == 4 and int((ref["next_token"] >= 0).sum()) > 0
        cases.append((call, ref))
    errors = []

    def worker(idx):
        try:
            torch.cuda.set_device(0)
            stream = torch.cuda.Stream()
            call, ref = cases[idx]
            with torch.cuda.stream(stream):
                for it in range(40):
                    out = call(stream=stream)
                    if it % 8 == 7:
                        stream.synchronize()
                        for k, v in ref.items():
                            if torch.is_tensor(v):
                                x, y = (v.view(torch.int32), out[k].view(torch.int32)) if v.dtype == torch.float32 else (v, out[k])
                                if not torch.equal(x, y):
                                    errors.append((idx, it, k))
                stream.synchronize()
                if psd.last_status() != psd.OK:
                    errors.append((idx, "status"))
            psd.release_stream(stream)      # the library keeps scratch for sixteen streams per device
        except Exception as e:   # noqa: BLE001
            errors.append((idx, repr(e)))

    threads = [threading.Thread(target=worker, args=(i,)) for i in range(2)]
    for th in threads:
        th.start()
    for th in threads:
        th.join()
    assert not errors, errors[:5]


def test_three_launch_form_replayed_from_a_cuda_graph(psd, wl):
    """The statistics launch and the three dependent finalisation launches captured into a CUDA graph (after two
    calls on the capturing stream, which size the library's buffers): replays on new contents of the same input
    buffers return what eager calls return."""
    dev = torch.device("cuda:0")
    B, K_d, K_q, V = 40, 6, 4, 16384
    rounds = [[x.to(dev) for x in wl.make_pyramid_inputs(B, K_d, K_q, V, "bf16", seed=140 + i, sigma_q=0.4, sigma_d=0.8)]
              for i in range(3)]
    probe = psd.verify_ex(*rounds[0], 1e9, 1e9)
    tau_q, tau_t = float(probe["div_q"].median()), float(probe["div_t"].median())
    psd.set_two_stage_policy(psd.TWO_STAGE_FUSED)
    try:
        eager = []
        for r in rounds:
            n0 = psd.launch_count()
            eager.append(psd.verify(*r, tau_q, tau_t, psd.FUZZY, 11, 4))
            torch.cuda.synchronize()
            assert psd.launch_count() - n0 == 4
        assert len({tuple(e["next_token"].tolist()) for e in eager}) == 3
        bufs = [t.clone() for t in rounds[0]]
        out = {k: torch.empty(B, dtype=torch.int32, device=dev) for k in ("accept_len_q", "next_token_q", "accept_len", "next_token")}
        side = torch.cuda.Stream()
        side.wait_stream(torch.cuda.current_stream())
        g = torch.cuda.CUDAGraph()
        try:
            with torch.cuda.stream(side):
                psd.set_stream()
                for _ in range(2):
                    psd.verify(*bufs, tau_q, tau_t, psd.FUZZY, 11, 4, out=out)
                side.synchronize()
                with torch.cuda.graph(g, stream=side):
                    psd.set_stream()
                    psd.verify(*bufs, tau_q, tau_t, psd.FUZZY, 11, 4, out=out)
        finally:
            psd.set_stream()
        for r, e in zip(rounds, eager):
            for dst, src in zip(bufs, r):
                dst.copy_(src)
            torch.cuda.synchronize()
            g.replay()
            torch.cuda.synchronize()
            for k in out:
                assert torch.equal(out[k], e[k]), k
        del g
        psd.release_stream(side)            # the graph is gone: nothing uses the stream's scratch any more
    finally:
        psd.set_two_stage_policy(psd.TWO_STAGE_DEFAULT)
    assert psd.last_status() == 0
