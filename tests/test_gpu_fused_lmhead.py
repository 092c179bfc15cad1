"""GPU parity of the fused LM-head path: logits = hidden x W^T computed by the tensor-core kernel and
consumed in its epilogue, against the oracle's double-precision GEMM followed by the ordinary stage."""
import numpy as np
import pytest
import torch

from parity_utils import TIE_DIV, TOL, host_bits

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def psd():
    if not torch.cuda.is_available():
        pytest.skip("no CUDA device")
    from paper_2510_12966_b200 import binding
    binding.load_library()
    torch.cuda.set_device(0)
    return binding


def make_case(B, K, d, V, seed, sigma_q=0.7, w_scale=0.02):
    g = torch.Generator().manual_seed(seed)
    h = torch.randn((B * K, d), generator=g).to(torch.bfloat16)
    w_t = (torch.randn((V, d), generator=g) * w_scale).to(torch.bfloat16)     # LM-head weight, out x in
    z = h.float() @ w_t.float().T
    z_q = (z + torch.randn((B * K, V), generator=g) * sigma_q).to(torch.bfloat16).reshape(B, K, V).contiguous()
    tok = torch.multinomial(torch.softmax(z_q.float().reshape(B * K, V), -1), 1, generator=g).reshape(B, K).to(torch.int32)
    return h.contiguous(), w_t.contiguous(), z_q, tok.contiguous()


def run_both(psd, oracle, h, w_t, z_q, tok, tau, mode, seed=3, offset=5, tile_variant=None, div_kind=0, want_resid=None):
    dev = torch.device("cuda:0")
    out = psd.verify_fused_lmhead(h.to(dev), w_t.to(dev), z_q.to(dev), tok.to(dev), tau, mode, seed, offset,
                                  tile_variant=tile_variant, div_kind=div_kind, want_resid=want_resid)
    torch.cuda.synchronize()
    assert psd.last_status() == 0
    gpu = {k: v.cpu().numpy() for k, v in out.items() if isinstance(v, torch.Tensor)}
    B, K, V = z_q.shape
    z = oracle.lmhead_logits(host_bits(h), host_bits(w_t.T.contiguous()), n_threads=16).reshape(B, K, V)
    orc = oracle.verify_stage_mixed(host_bits(z_q), z, tok.numpy(), np.float32(tau), mode, seed, offset, div_kind=div_kind,
                                    n_threads=16)
    orc["z_large"], orc["z_small"], orc["tokens"], orc["seed"], orc["offset"] = z, host_bits(z_q), tok.numpy(), seed, offset
    return gpu, orc


def classify_mismatch(oracle, gpu, orc, b, tau, mode, gid=None):
    """A sequence whose integers differ from the oracle's must be one of the counted near ties of the logits path,
    judged on the oracle's own double-precision quantities (the fused path is in the bf16 tolerance class: its
    large logits come out of a tensor-core sum over d_model in single precision, its small logits are bf16):
    accept length -- |D - tau| < 1e-4 or |u - min(1, rho)| < 2e-3 at the first differing position; token -- the
    GPU's token has positive weight and the oracle's target lies within 1e-4 of the total weight of the
    prefix-sum boundary between the two tokens, with less than that between them. Returns the class."""
    tol = TOL["bf16"]
    K = orc["div"].shape[1]
    gid = b if gid is None else gid
    Lg, Lo = int(gpu["accept_len"][b]), int(orc["accept_len"][b])
    k = min(Lg, Lo)
    p, _ = oracle.softmax(orc["z_large"][b, min(k, K - 1)])
    q, _ = oracle.softmax(orc["z_small"][b, min(k, K - 1)])
    u, u2 = oracle.row_uniforms(orc["seed"], orc["offset"], gid * K + min(k, K - 1))
    if Lg != Lo:
        x = int(orc["tokens"][b, k])
        rho = (p[x] / q[x]) if q[x] > 0 else (np.inf if p[x] > 0 else 0.0)
        tie_d = mode in (0, 2) and abs(orc["div"][b, k] - tau) < TIE_DIV
        tie_c = mode in (1, 2, 3) and abs(u - min(1.0, rho)) < tol["coin"]
        assert tie_d or tie_c, (f"seq {b} pos {k}: accept_len gpu {Lg} oracle {Lo}, D={orc['div'][b, k]} tau={tau} "
                                f"u={u} rho={rho} -- not a near tie")
        return "tie_div" if tie_d else "tie_coin"
    tg, to = int(gpu["next_token"][b]), int(orc["next_token"][b])
    assert Lo < K and tg >= 0 and to >= 0, f"seq {b}: next_token gpu {tg} oracle {to}"
    w = np.maximum(p - q, 0.0)
    if mode == 3 or not (orc["resid_mass"][b, Lo] > 0):
        w = p
    c = np.cumsum(w)
    target = u2 * c[-1]
    lo, hi = min(tg, to), max(tg, to)
    margin = abs(c[lo] - target) / c[-1]
    between = (c[hi - 1] - c[lo]) / c[-1] if hi - 1 > lo else 0.0
    assert w[tg] > 0, f"seq {b}: gpu token {tg} has zero weight"
    assert margin < tol["cdf"] and between < tol["cdf"], (
        f"seq {b} row {Lo}: token gpu {tg} oracle {to}, margin {margin:.3e}, between {between:.3e} of W -- not a near tie")
    return "tie_cdf"


def check(oracle, gpu, orc, tau, mode, max_token_ties=1):
    fin = np.isfinite(orc["div"])
    assert np.abs(gpu["div"][fin] - orc["div"][fin]).max() < 2e-3, np.abs(gpu["div"][fin] - orc["div"][fin]).max()
    assert np.all(np.isinf(gpu["div"][np.isinf(orc["div"])]))
    if "resid_mass" in gpu:
        assert np.abs(gpu["resid_mass"] - orc["resid_mass"]).max() < 2e-3
    ties = 0
    for b in range(len(orc["accept_len"])):
        if int(gpu["accept_len"][b]) == int(orc["accept_len"][b]) and int(gpu["next_token"][b]) == int(orc["next_token"][b]):
            continue
        classify_mismatch(oracle, gpu, orc, b, float(np.float32(tau)), mode)
        ties += 1
    assert ties <= max_token_ties, ties
    return ties


@pytest.mark.parametrize("B,K,d,V", [(2, 4, 128, 1000), (3, 5, 256, 4099), (32, 8, 512, 2048)])
def test_fused_lmhead_small_shapes(psd, oracle, B, K, d, V):
    """Ragged last tile (V not a multiple of 128), fewer rows than the 256-row tile, several K steps."""
    h, w_t, z_q, tok = make_case(B, K, d, V, seed=50 + V, w_scale=0.08)
    for tau, mode in ((0.05, 0), (0.2, 0), (0.0, 1)):
        gpu, orc = run_both(psd, oracle, h, w_t, z_q, tok, tau, mode)
        check(oracle, gpu, orc, tau, mode)
        assert 0 <= orc["accept_len"].sum() <= B * K


def test_fused_lmhead_reduced_cfg5(psd, oracle):
    """workload configuration 5 recipe (B=32, K=8, d=4096, W ~ N(0, 0.02^2), qualifier noise 0.7) at V=4096."""
    h, w_t, z_q, tok = make_case(32, 8, 4096, 4096, seed=5000)
    gpu, orc = run_both(psd, oracle, h, w_t, z_q, tok, 0.2, 0)       # the config's threshold: accepts everything here
    check(oracle, gpu, orc, 0.2, 0, max_token_ties=2)
    tau = float(np.float32(np.median(orc["div"])))                    # a threshold that splits the rows
    gpu, orc = run_both(psd, oracle, h, w_t, z_q, tok, tau, 0)
    check(oracle, gpu, orc, tau, 0, max_token_ties=3)
    assert 0 < orc["accept_len"].sum() < 32 * 8
    gpu, orc = run_both(psd, oracle, h, w_t, z_q, tok, 0.0, 1)        # strict mode: coin flips on token probabilities
    check(oracle, gpu, orc, 0.0, 1, max_token_ties=3)


def test_fused_lmhead_full_size_cfg5_sampled(psd, oracle):
    """workload configuration 5 at full size (M=256, d=4096, V=128256) in the launch configuration bench.py times,
    at the config's threshold and at one that splits the rows; the oracle recomputes three sampled sequences (its
    double-precision GEMM is far too slow for all 256 rows) and every one of them is checked down to the token."""
    from paper_2510_12966_b200 import workloads
    dev = torch.device("cuda:0")
    w = workloads.CONFIGS[5]
    h, w_t, z_q, tok = workloads.make_fused_inputs(w.B, w.K_d, w.V, w.d_model, seed=5000, sigma_q=w.sigma_q, device=dev)
    w_host = host_bits(w_t.T.contiguous())
    pick = (0, 17, 31)
    z_orc = {b: oracle.lmhead_logits(host_bits(h[b * w.K_d:(b + 1) * w.K_d]), w_host, n_threads=16).reshape(1, w.K_d, w.V)
             for b in pick}
    tau_split, rejected, ties = None, 0, 0
    for tau in (w.tau_t, None):
        tau = tau_split if tau is None else tau
        out = psd.verify_fused_lmhead(h, w_t, z_q, tok, tau, psd.FUZZY, 0, 0)
        torch.cuda.synchronize()
        assert psd.last_status() == 0
        div, resid = out["div"].cpu().numpy(), out["resid_mass"].cpu().numpy()
        al, nt = out["accept_len"].cpu().numpy(), out["next_token"].cpu().numpy()
        assert np.all(np.isfinite(div)) and np.all((div >= 0) & (div <= 0.6932))
        assert np.all((0 <= al) & (al <= w.K_d)) and np.all((nt >= 0) == (al < w.K_d)) and np.all(nt < w.V)
        tau_split = float(np.float32(np.median(div)))
        for b in pick:
            z = z_orc[b]
            # the oracle sees a batch of one; fuzzy accept bits use no uniform, and the draw is redone below with the
            # Philox block of the row's index in the full batch
            orc = oracle.verify_stage_mixed(host_bits(z_q[b:b + 1]), z, tok[b:b + 1].cpu().numpy(), np.float32(tau),
                                            oracle.FUZZY, 0, 0, n_threads=16)
            assert np.abs(div[b] - orc["div"][0]).max() < 2e-3
            assert np.abs(resid[b] - orc["resid_mass"][0]).max() < 2e-3
            orc.update(z_large=z, z_small=host_bits(z_q[b:b + 1]), tokens=tok[b:b + 1].cpu().numpy(), seed=0, offset=0)
            Lo = int(orc["accept_len"][0])
            if Lo < w.K_d:
                rejected += 1
                p, _ = oracle.softmax(z[0, Lo])
                q, _ = oracle.softmax(host_bits(z_q[b, Lo]))
                wts = np.maximum(p - q, 0.0) if orc["resid_mass"][0, Lo] > 0 else p
                _, u2 = oracle.row_uniforms(0, 0, b * w.K_d + Lo)
                orc["next_token"][0] = oracle.inverse_cdf(wts, u2)
            if al[b] != Lo or nt[b] != orc["next_token"][0]:
                classify_mismatch(oracle, dict(accept_len=al[b:b + 1], next_token=nt[b:b + 1]), orc, 0, float(np.float32(tau)), 0, gid=b)
                ties += 1
    assert rejected >= 2 and ties <= 1


def test_fused_lmhead_one_sm_variant_agrees(psd, oracle):
    """The one-SM sweeps (tile_variant = PSD_LMHEAD_TILES_ONE_SM) against the oracle, so that both variants stay covered."""
    h, w_t, z_q, tok = make_case(32, 8, 512, 2048, seed=61, w_scale=0.08)
    gpu, orc = run_both(psd, oracle, h, w_t, z_q, tok, 0.1, 0, tile_variant=psd.LMHEAD_TILES_ONE_SM)
    check(oracle, gpu, orc, 0.1, 0)
    gpu2, _ = run_both(psd, oracle, h, w_t, z_q, tok, 0.1, 0)
    assert np.array_equal(gpu["accept_len"], gpu2["accept_len"])


@pytest.mark.parametrize("tile_variant", [None, 1])
def test_fused_lmhead_kl_single_sweep(psd, oracle, tile_variant):
    """KL(large || small): the divergences come out of the first GEMM sweep; the second one only serves residual masses.
    Threshold mode with a threshold that splits the rows (rejected rows draw from the residual: the second sweep runs),
    the same without the residual output, everything accepted (no draw: it returns at once), the assisted mode (draws
    from p_large off the first sweep's tile sums), strict mode, and a masked small logit under a live large one
    (divergence +inf). Two row blocks, ragged last tile."""
    KL = 2
    h, w_t, z_q, tok = make_case(40, 8, 256, 1500, seed=88, w_scale=0.08)
    probe, orc = run_both(psd, oracle, h, w_t, z_q, tok, 1e9, 0, div_kind=KL, tile_variant=tile_variant)
    check(oracle, probe, orc, 1e9, 0)
    assert np.all(probe["accept_len"] == 8) and np.all(probe["next_token"] == -1)
    gpu, orc = run_both(psd, oracle, h, w_t, z_q, tok, 1e9, 0, div_kind=KL, want_resid=False, tile_variant=tile_variant)   # one sweep
    check(oracle, gpu, orc, 1e9, 0)
    assert np.array_equal(gpu["div"], probe["div"])
    tau = float(np.float32(np.median(orc["div"])))
    for want_resid in (True, False):
        gpu, orc = run_both(psd, oracle, h, w_t, z_q, tok, tau, 0, div_kind=KL, want_resid=want_resid, tile_variant=tile_variant)
        check(oracle, gpu, orc, tau, 0, max_token_ties=3)
        assert 0 < orc["accept_len"].sum() < 40 * 8 and np.all((gpu["next_token"] >= 0) == (gpu["accept_len"] < 8))
    gpu, orc = run_both(psd, oracle, h, w_t, z_q, tok, 0.0, 3, div_kind=KL, want_resid=False, tile_variant=tile_variant)   # assisted
    check(oracle, gpu, orc, 0.0, 3, max_token_ties=3)
    assert 0 < orc["accept_len"].sum() < 40 * 8
    gpu, orc = run_both(psd, oracle, h, w_t, z_q, tok, 0.0, 1, div_kind=KL, want_resid=False, tile_variant=tile_variant)   # strict
    check(oracle, gpu, orc, 0.0, 1, max_token_ties=3)
    z_q[3, 2, 700:760] = -float("inf")
    gpu, orc = run_both(psd, oracle, h, w_t, z_q, tok, tau, 0, div_kind=KL, tile_variant=tile_variant)
    assert np.isinf(orc["div"][3, 2]) and np.isinf(gpu["div"][3, 2]) and gpu["accept_len"][3] <= 2
    check(oracle, gpu, orc, tau, 0, max_token_ties=3)
    dev = torch.device("cuda:0")
    bad = psd.verify_fused_lmhead(h.to(dev), w_t.to(dev), z_q.to(dev), tok.to(dev), 0.1, div_kind=1, raise_on_error=False)
    assert bad["status"] == psd.ERR_UNSUPPORTED          # total variation does not separate: no fused form


def test_fused_lmhead_more_than_one_row_block(psd, oracle):
    """B*K = 40*8 = 320 rows: two blocks of 256 rows (the second one partial)."""
    h, w_t, z_q, tok = make_case(40, 8, 256, 1536, seed=77, w_scale=0.08)
    gpu, orc = run_both(psd, oracle, h, w_t, z_q, tok, 0.08, 0)
    check(oracle, gpu, orc, 0.08, 0, max_token_ties=2)
    tau = float(np.float32(np.median(orc["div"])))      # a threshold that splits the rows, in both blocks
    gpu, orc = run_both(psd, oracle, h, w_t, z_q, tok, tau, 0)
    check(oracle, gpu, orc, tau, 0, max_token_ties=3)
    assert 0 < orc["accept_len"][:32].sum() < 32 * 8 and 0 < orc["accept_len"][32:].sum() < 8 * 8


def test_fused_lmhead_masked_and_poisoned_rows(psd, oracle):
    """-inf in the small logits (masked vocabulary), a NaN in a hidden row, a token out of range."""
    h, w_t, z_q, tok = make_case(4, 4, 128, 1000, seed=78, w_scale=0.08)
    z_q[0, 1, 100:700] = -float("inf")
    h[2 * 4 + 1, 5] = float("nan")            # sequence 2, position 1: the large model's row is poisoned
    tok[3, 2] = 1000                           # out of range
    gpu, orc = run_both(psd, oracle, h, w_t, z_q, tok, 1.0, 0)
    assert gpu["accept_len"][2] == 1 and gpu["next_token"][2] == -2
    assert gpu["accept_len"][3] == 2 and gpu["next_token"][3] >= 0
    assert np.array_equal(gpu["accept_len"], orc["accept_len"])
    ok = np.isfinite(orc["div"])
    assert np.abs(gpu["div"][ok] - orc["div"][ok]).max() < 2e-3


def test_fused_lmhead_rejects_unsupported_shapes(psd):
    dev = torch.device("cuda:0")
    h2 = torch.zeros((8, 96), dtype=torch.bfloat16, device=dev)
    w2 = torch.zeros((512, 96), dtype=torch.bfloat16, device=dev)
    z2 = torch.zeros((1, 8, 512), dtype=torch.bfloat16, device=dev)
    t2 = torch.zeros((1, 8), dtype=torch.int32, device=dev)
    assert psd.verify_fused_lmhead(h2, w2, z2, t2, 0.1, raise_on_error=False)["status"] == psd.ERR_UNSUPPORTED  # d % 64
