"""The allocation-free entry point against the ordinary one.

`pyramidsd_verify_stage_noalloc` exists for callers that are not allowed to allocate device memory while
they run: a serving process that handed out all of its memory at start-up, a plug-in living inside
another program's memory plan. It keeps its per-row scratch in an array that is part of the library
image instead of a workspace. This file is collected last on purpose: if the new entry point were
broken, a run that stops at the first failure has already gone through every other test. The test
stands on its own (fresh process) and also after the rest of the suite, and it makes two calls in a row
because the built-in array is shared by all calls and keeps the previous call's contents.
"""
import numpy as np
import pytest
import torch

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def psd():
    if not torch.cuda.is_available():
        pytest.skip("no CUDA device")
    from paper_2510_12966_b200 import binding
    binding.load_library()
    torch.cuda.set_device(0)
    return binding


def _outputs(B, dev):
    return (torch.full((B,), -7, dtype=torch.int32, device=dev), torch.full((B,), -7, dtype=torch.int32, device=dev),
            torch.full((1,), -7, dtype=torch.int32, device=dev))


def test_noalloc_entry_point_matches_the_workspace_entry_point_twice_in_a_row(psd):
    from paper_2510_12966_b200 import workloads
    dev = torch.device("cuda:0")
    # two different stages back to back: the second one runs on scratch the first one has written to,
    # with fewer rows, another vocabulary size and another mode
    cases = [dict(B=12, K=8, V=32768, dtype="bf16", seed=901, tau=0.08, mode=psd.FUZZY, offset=3),
             dict(B=5, K=6, V=20000, dtype="f32", seed=902, tau=0.05, mode=psd.STRICT, offset=4)]
    for c in cases:
        zs, zl, tok = [t.to(dev) for t in workloads.make_stage_inputs(c["B"], c["K"], c["V"], c["dtype"], seed=c["seed"],
                                                                    sigma=0.7)]
        ref_len, ref_tok = psd.verify_stage(zs, zl, tok, c["tau"], c["mode"], 11, c["offset"])
        out_len, out_tok, flag = _outputs(c["B"], dev)     # outputs are the caller's; the entry point makes none
        rc = psd.verify_stage_noalloc(zs, zl, tok, c["tau"], c["mode"], 11, c["offset"], out_accept_len=out_len,
                                      out_next_token=out_tok, out_wait_timeout=flag)
        torch.cuda.synchronize()
        assert rc == psd.OK and flag.item() == 0
        # integer results: the tolerance of the parity tests is "bit-exact", and both paths run the same kernels
        assert torch.equal(out_len, ref_len), (out_len.tolist(), ref_len.tolist())
        assert torch.equal(out_tok, ref_tok), (out_tok.tolist(), ref_tok.tolist())
        assert 0 < int(ref_len.sum()) < c["B"] * c["K"]     # the case has both accepted and rejected positions
    assert psd.last_status() == 0


def test_noalloc_entry_point_rejects_stages_beyond_its_builtin_scratch(psd):
    dev = torch.device("cuda:0")
    B, K, V = psd.NOALLOC_MAX_ROWS // 32 + 1, 32, 2048      # one sequence too many
    z = torch.zeros((B, K, V), dtype=torch.bfloat16, device=dev)
    tok = torch.zeros((B, K), dtype=torch.int32, device=dev)
    out_len, out_tok, flag = _outputs(B, dev)
    rc = psd.verify_stage_noalloc(z, z, tok, 0.1, out_accept_len=out_len, out_next_token=out_tok, out_wait_timeout=flag,
                                  raise_on_error=False)
    torch.cuda.synchronize()
    assert rc == psd.ERR_UNSUPPORTED
    assert np.all(out_len.cpu().numpy() == -7) and flag.item() == -7      # nothing was launched
    # the largest stage it takes still runs
    B = psd.NOALLOC_MAX_ROWS // 32
    out_len, out_tok, flag = _outputs(B, dev)
    rc = psd.verify_stage_noalloc(z[:B], z[:B], tok[:B], 0.1, out_accept_len=out_len, out_next_token=out_tok,
                                  out_wait_timeout=flag)
    torch.cuda.synchronize()
    assert rc == psd.OK and flag.item() == 0 and np.all(out_len.cpu().numpy() == 32)


def test_noalloc_entry_point_as_the_first_call_of_a_process_allocates_nothing(oracle):
    """A fresh process whose first and only library calls are the allocation-free entry point: it works without any
    earlier call having set the library up, the free device memory is the same before and after the calls (loading
    the kernels themselves, which the driver does on the first launch, is taken out by a warm-up call), and the
    results equal the oracle's. The second shape has an odd vocabulary size, so the kernel that takes every shape
    runs on the built-in array as well as the cluster kernel."""
    import os, subprocess, sys, textwrap
    if not torch.cuda.is_available():
        pytest.skip("no CUDA device")
    root = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
    code = textwrap.dedent("""
        import sys, numpy as np, torch
        sys.path.insert(0, %r); sys.path.insert(0, %r)
        import oracle
        from paper_2510_12966_b200 import binding as psd, workloads as wl
        from parity_utils import compare_stage, host_bits
        torch.cuda.set_device(0)
        dev = torch.device("cuda:0")
        psd.load_library()
        cases = [dict(B=6, K=5, V=16384, dtype="bf16", seed=911, tau=0.08, mode=psd.FUZZY),
                 dict(B=4, K=3, V=5001, dtype="f32", seed=912, tau=0.05, mode=psd.STRICT)]
        data = []
        for c in cases:
            zs, zl, tok = wl.make_stage_inputs(c["B"], c["K"], c["V"], c["dtype"], seed=c["seed"], sigma=0.7)
            outs = [torch.full((c["B"],), -7, dtype=torch.int32, device=dev) for _ in range(2)] + [torch.full((1,), -7, dtype=torch.int32, device=dev)]
            data.append((c, zs, zl, tok, zs.to(dev), zl.to(dev), tok.to(dev), outs))
        def call(d):
            c, _, _, _, zs, zl, tok, outs = d
            return psd.verify_stage_noalloc(zs, zl, tok, c["tau"], c["mode"], 11, 3, out_accept_len=outs[0], out_next_token=outs[1],
                                            out_wait_timeout=outs[2])
        for d in data:                      # the very first library calls of this process; they also load the kernels
            assert call(d) == psd.OK
        torch.cuda.synchronize()
        free0, _ = torch.cuda.mem_get_info()
        for _ in range(3):
            for d in data:
                assert call(d) == psd.OK
        torch.cuda.synchronize()
        free1, _ = torch.cuda.mem_get_info()
        assert free0 == free1, (free0, free1)
        for c, zs, zl, tok, _, _, _, outs in data:
            assert outs[2].item() == 0
            gpu = dict(accept_len=outs[0].cpu().numpy(), next_token=outs[1].cpu().numpy())
            orc = oracle.verify_stage(host_bits(zs), host_bits(zl), tok.numpy(), np.float32(c["tau"]), c["mode"], 11, 3, n_threads=4)
            rep = compare_stage(oracle, gpu, orc, host_bits(zs), host_bits(zl), dtype=c["dtype"], mode=c["mode"],
                                tau=float(np.float32(c["tau"])), seed=11, offset=3, check_rows=False)
            assert rep["tie_div"] + rep["tie_coin"] + rep["tie_cdf"] <= 1
            assert 0 < int(orc["accept_len"].sum()) < c["B"] * c["K"]
        print("ok")
    """) % (root, os.path.join(root, "tests"))
    run = subprocess.run([sys.executable, "-c", code], capture_output=True, text=True, timeout=600)
    assert run.returncode == 0 and "ok" in run.stdout, (run.stdout[-1000:], run.stderr[-3000:])
