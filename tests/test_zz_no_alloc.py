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
