"""Pins for the CPU oracle: each test ties one piece of it to something outside itself — published
known-answer vectors, hand-computed values, closed forms, library routines on special cases, exhaustive
enumeration, or a Monte Carlo check of the distribution the method must reproduce."""
import itertools
import math
import os

import numpy as np
import pytest
from scipy import stats
from scipy.spatial.distance import jensenshannon
from scipy.special import rel_entr, softmax as sp_softmax

GOLDEN = os.path.join(os.path.dirname(__file__), "golden")
LN2 = math.log(2.0)


def _rows(path):
    with open(path) as f:
        return [ln.strip() for ln in f if ln.strip() and not ln.startswith("#")]


# ---------------------------------------------------------------- Philox4x32-10
def test_philox_known_answers(oracle):
    for ln in _rows(os.path.join(GOLDEN, "philox4x32_10_kat.txt")):
        w = [int(x, 16) for x in ln.split()]
        out = oracle.philox4x32_10(w[0:4], w[4:6])
        assert [int(x) for x in out] == w[6:10], ln


def test_row_uniforms_use_counter_layout(oracle):
    # counter = (row, 0, offset_lo, offset_hi), key = (seed_lo, seed_hi); u from word 0, u2 from word 1
    seed, offset, row = 0x0123456789ABCDEF, 0xFEDCBA9876543210, 77
    w = oracle.philox4x32_10([row, 0, offset & 0xFFFFFFFF, offset >> 32], [seed & 0xFFFFFFFF, seed >> 32])
    u, u2 = oracle.row_uniforms(seed, offset, row)
    assert u == (int(w[0]) >> 8) / 2.0**24 and u2 == (int(w[1]) >> 8) / 2.0**24
    assert 0.0 <= u < 1.0 and np.float32(u) == u  # exactly representable in fp32


def test_uniforms_are_uniform(oracle):
    us = np.array([oracle.row_uniforms(3, 5, r) for r in range(20000)])
    for col in (0, 1):
        assert stats.kstest(us[:, col], "uniform").pvalue > 1e-3
    assert abs(np.corrcoef(us[:, 0], us[:, 1])[0, 1]) < 0.03


# ---------------------------------------------------------------- softmax
def test_softmax_matches_library_and_is_shift_invariant(oracle):
    rng = np.random.default_rng(0)
    z = rng.normal(0, 3, 257)
    p, ok = oracle.softmax(z)
    assert ok and abs(p.sum() - 1.0) < 1e-12
    np.testing.assert_allclose(p, sp_softmax(z), rtol=1e-12, atol=0)
    p2, _ = oracle.softmax(z + 123.0)
    np.testing.assert_allclose(p2, p, rtol=1e-10)
    p3, _ = oracle.softmax(z, inv_temperature=1 / 0.7)
    np.testing.assert_allclose(p3, sp_softmax(z / 0.7), rtol=1e-12)


def test_softmax_masked_and_invalid_rows(oracle):
    z = np.array([0.0, -np.inf, 1.0, -np.inf])
    p, ok = oracle.softmax(z)
    assert ok and p[1] == 0.0 and p[3] == 0.0 and abs(p.sum() - 1) < 1e-15
    for bad in (np.nan, np.inf):
        _, ok = oracle.softmax(np.array([0.0, bad, 1.0]))
        assert not ok
    _, ok = oracle.softmax(np.full(5, -np.inf))
    assert not ok


def test_softmax_bf16_and_f32_inputs_are_read_exactly(oracle):
    # bf16 bit pattern 0x4049 = 3.140625, 0xC000 = -2.0
    bits = np.array([0x4049, 0xC000, 0x0000], dtype=np.uint16)
    p, _ = oracle.softmax(bits)
    np.testing.assert_allclose(p, sp_softmax(np.array([3.140625, -2.0, 0.0])), rtol=1e-14)
    z32 = np.array([0.1, 0.2, 0.3], dtype=np.float32)
    p, _ = oracle.softmax(z32)
    np.testing.assert_allclose(p, sp_softmax(z32.astype(np.float64)), rtol=1e-14)


# ---------------------------------------------------------------- divergence
def test_divergence_hand_cases(oracle):
    for ln in _rows(os.path.join(GOLDEN, "divergence_hand_cases.txt")):
        name, p, q, js, tv, kl = [s.strip() for s in ln.split("|")]
        p = np.array(p.split(), float)
        q = np.array(q.split(), float)
        assert abs(oracle.divergence(p, q, oracle.JS) - float(js)) < 5e-10, name
        assert abs(oracle.divergence(p, q, oracle.TV) - float(tv)) < 5e-10, name
        assert abs(oracle.divergence(p, q, oracle.KL) - float(kl)) < 5e-10, name
        assert abs(oracle.residual_mass(p, q) - float(tv)) < 5e-10, name


def test_divergence_logits_case(oracle):
    p, _ = oracle.softmax(np.array([2.0, 1.0, 0.0, -1.0]))
    q, _ = oracle.softmax(np.ones(4))
    np.testing.assert_allclose(p, [0.6439142599, 0.2368828181, 0.0871443187, 0.0320586033], atol=5e-11)
    assert abs(oracle.divergence(p, q, oracle.JS) - 0.1133397211) < 5e-10
    assert abs(oracle.residual_mass(p, q) - 0.3939142599) < 5e-10


def test_divergence_against_library_routines(oracle):
    rng = np.random.default_rng(1)
    for V in (2, 3, 17, 1000):
        p = sp_softmax(rng.normal(0, 3, V))
        q = sp_softmax(rng.normal(0, 3, V))
        js = oracle.divergence(p, q, oracle.JS)
        assert abs(js - jensenshannon(p, q) ** 2) < 1e-12
        assert abs(oracle.divergence(p, q, oracle.KL) - rel_entr(p, q).sum()) < 1e-12
        tv = oracle.divergence(p, q, oracle.TV)
        assert abs(tv - 0.5 * np.abs(p - q).sum()) < 1e-14
        # invariants: bounded, symmetric, residual mass equals total variation, Lin's bound JS <= ln2 * TV
        assert 0.0 <= js <= LN2
        assert abs(js - oracle.divergence(q, p, oracle.JS)) < 1e-14
        assert abs(oracle.residual_mass(p, q) - tv) < 1e-13
        assert js <= LN2 * tv + 1e-15
    # KL is NOT symmetric: a transposed operand order must show
    p, q = np.array([0.9, 0.1]), np.array([0.5, 0.5])
    assert abs(oracle.divergence(p, q, oracle.KL) - (0.9 * math.log(1.8) + 0.1 * math.log(0.2))) < 1e-14


def test_divergence_degenerate_cases(oracle):
    p = np.array([0.1, 0.2, 0.3, 0.4])
    assert oracle.divergence(p, p, oracle.JS) == 0.0
    assert oracle.residual_mass(p, p) == 0.0
    a, b = np.array([1.0, 0.0]), np.array([0.0, 1.0])
    assert abs(oracle.divergence(a, b, oracle.JS) - LN2) < 1e-15
    assert oracle.divergence(a, b, oracle.TV) == 1.0
    assert oracle.divergence(a, b, oracle.KL) == math.inf
    for V in (2, 8, 100):
        onehot = np.zeros(V)
        onehot[V // 2] = 1.0
        uni = np.full(V, 1.0 / V)
        closed = 0.5 * math.log(2 * V / (V + 1)) + 0.5 * ((1 / V) * math.log(2 / (V + 1)) + ((V - 1) / V) * LN2)
        assert abs(oracle.divergence(onehot, uni, oracle.JS) - closed) < 1e-13
        assert abs(oracle.divergence(onehot, uni, oracle.TV) - (1 - 1 / V)) < 1e-14
    assert abs(0.4969291266 - (0.5 * math.log(16 / 9) + 0.5 * ((1 / 8) * math.log(2 / 9) + (7 / 8) * LN2))) < 1e-10


# ---------------------------------------------------------------- prefix scan, inverse CDF
def test_prefix_length_exhaustive(oracle):
    for K in range(0, 11):
        for bits in itertools.product((0, 1), repeat=K):
            mask = sum(b << i for i, b in enumerate(bits))
            inv = ~mask & ((1 << K) - 1)
            expect = K if inv == 0 else (inv & -inv).bit_length() - 1  # ffs(~mask)
            assert oracle.prefix_length(bits, K) == expect
    assert oracle.prefix_length([1, 1, 1, 0], 2) == 2  # only the first n_valid positions count
    assert oracle.prefix_length([0, 1, 1], 3) == 0


def test_inverse_cdf_enumeration(oracle):
    rng = np.random.default_rng(2)
    for V in (2, 3, 5, 8):
        w = rng.integers(0, 4, V).astype(float)  # some weights are exactly zero
        w[rng.integers(0, V)] += 1.0
        n = 256
        picks = np.array([oracle.inverse_cdf(w, j / n) for j in range(n)])
        hist = np.bincount(picks, minlength=V) / n
        assert np.all(np.abs(hist - w / w.sum()) <= 1.0 / n + 1e-12)
        assert np.all(hist[w == 0] == 0)            # zero-weight tokens are never emitted
        assert np.all(np.diff(picks) >= 0)          # monotone in u
    assert oracle.inverse_cdf(np.array([0.25, 0.25, 0.5]), 0.25) == 1   # inclusive prefix must EXCEED u*W
    assert oracle.inverse_cdf(np.array([0.25, 0.25, 0.5]), 0.0) == 0
    assert oracle.inverse_cdf(np.array([0.0, 0.0, 1.0, 0.0]), 0.999999) == 2
    assert oracle.inverse_cdf(np.zeros(4), 0.5) == -1


# ---------------------------------------------------------------- one stage
def _logits_from_probs(p):
    with np.errstate(divide="ignore"):
        return np.log(np.asarray(p, float))


def test_stage_three_point_hand_case(oracle):
    # p_large = (0.6, 0.3, 0.1), p_small = (0.2, 0.5, 0.3): JS = 0.0911..., residual (0.4, 0, 0) -> token 0
    zl = _logits_from_probs([0.6, 0.3, 0.1]).reshape(1, 1, 3)
    zs = _logits_from_probs([0.2, 0.5, 0.3]).reshape(1, 1, 3)
    for off in range(50):
        out = oracle.verify_stage(zs, zl, [[1]], tau=0.05, offset=off)
        assert out["accept_len"][0] == 0 and out["next_token"][0] == 0
    out = oracle.verify_stage(zs, zl, [[1]], tau=0.0912)
    assert out["accept_len"][0] == 1 and out["next_token"][0] == -1
    assert abs(out["div"][0, 0] - 0.0911207985) < 5e-10
    assert abs(out["p_large_tok"][0, 0] - 0.3) < 1e-12 and abs(out["p_small_tok"][0, 0] - 0.5) < 1e-12
    assert abs(out["resid_mass"][0, 0] - 0.4) < 1e-12


def test_fuzzy_threshold_properties(oracle):
    rng = np.random.default_rng(3)
    B, K, V = 6, 5, 64
    zl = rng.normal(0, 3, (B, K, V))
    zs = zl + rng.normal(0, 1, (B, K, V))
    tok = rng.integers(0, V, (B, K))
    none = oracle.verify_stage(zs, zl, tok, tau=-1e-9)
    assert np.all(none["accept_len"] == 0) and np.all(none["next_token"] >= 0)
    full = oracle.verify_stage(zs, zl, tok, tau=np.float32(LN2) + 1e-6)
    assert np.all(full["accept_len"] == K) and np.all(full["next_token"] == -1)
    prev = -1
    for tau in (0.0, 0.05, 0.1, 0.2, 0.3, 0.5, 0.7):
        out = oracle.verify_stage(zs, zl, tok, tau=tau)
        n = int(out["accept_bits"].sum())
        assert n >= prev
        prev = n
        # accept bit is exactly D <= tau, prefix length follows the bits
        assert np.array_equal(out["accept_bits"], (out["div"] <= tau).astype(np.int32))
        for b in range(B):
            assert out["accept_len"][b] == oracle.prefix_length(out["accept_bits"][b], K)
    same = oracle.verify_stage(zl, zl, tok, tau=0.0)  # identical rows: D == 0 exactly, accepted at tau = 0
    assert np.all(same["div"] == 0.0) and np.all(same["accept_len"] == K)


def test_resample_never_emits_zero_residual_token(oracle):
    rng = np.random.default_rng(4)
    V = 12
    zl = rng.normal(0, 2, (1, 1, V))
    zs = rng.normal(0, 2, (1, 1, V))
    p, _ = oracle.softmax(zl.ravel())
    q, _ = oracle.softmax(zs.ravel())
    for off in range(400):
        out = oracle.verify_stage(zs, zl, [[0]], tau=-1.0, offset=off)
        t = out["next_token"][0]
        assert p[t] > q[t]


def _emitted_distribution(oracle, p, q, mode, n, seed):
    """Draw x ~ q n times, run one strict/assisted verification per draw, return emitted-token counts."""
    V = len(p)
    rng = np.random.default_rng(seed)
    x = rng.choice(V, size=n, p=q).astype(np.int32)
    zl = np.broadcast_to(_logits_from_probs(p), (n, 1, V)).copy()
    zs = np.broadcast_to(_logits_from_probs(q), (n, 1, V)).copy()
    out = oracle.verify_stage(zs, zl, x.reshape(n, 1), tau=0.0, mode=mode, seed=seed, offset=17, n_threads=8)
    emitted = np.where(out["accept_len"] == 1, x, out["next_token"])
    return np.bincount(emitted, minlength=V), out["accept_len"].mean()


def test_strict_mode_reproduces_target_distribution(oracle):
    # Standard speculative sampling must emit tokens distributed exactly as the larger model's p.
    rng = np.random.default_rng(5)
    V, n = 16, 1_000_000
    p = sp_softmax(rng.normal(0, 1.5, V))
    q = sp_softmax(rng.normal(0, 1.5, V))
    counts, acc_rate = _emitted_distribution(oracle, p, q, oracle.STRICT, n, seed=11)
    chi = stats.chisquare(counts, p * n)
    assert chi.pvalue > 1e-3, chi
    tv = 0.5 * np.abs(p - q).sum()
    sigma = math.sqrt(tv * (1 - tv) / n)
    assert abs(acc_rate - (1 - tv)) < 4 * sigma
    # the same statistic must reject a wrong target (power check: the draft distribution q)
    assert stats.chisquare(counts, q * n).pvalue < 1e-6


def test_assisted_mode_emits_min_plus_reject_mass_times_p(oracle):
    # Sec. 3.4: on rejection the assisted variant samples from the larger model directly, so the
    # emitted law is min(p, q) + (1 - sum min(p, q)) * p.
    rng = np.random.default_rng(6)
    V, n = 16, 400_000
    p = sp_softmax(rng.normal(0, 1.5, V))
    q = sp_softmax(rng.normal(0, 1.5, V))
    counts, _ = _emitted_distribution(oracle, p, q, oracle.ASSISTED, n, seed=12)
    law = np.minimum(p, q) + (1 - np.minimum(p, q).sum()) * p
    assert stats.chisquare(counts, law * n).pvalue > 1e-3
    assert stats.chisquare(counts, p * n).pvalue < 1e-6


def test_fallback_mode_with_negative_tau_equals_strict(oracle):
    rng = np.random.default_rng(7)
    B, K, V = 8, 6, 50
    zl = rng.normal(0, 2, (B, K, V)).astype(np.float32)
    zs = (zl + rng.normal(0, 0.7, (B, K, V))).astype(np.float32)
    tok = rng.integers(0, V, (B, K))
    a = oracle.verify_stage(zs, zl, tok, tau=-1.0, mode=oracle.FUZZY_SD_FALLBACK, seed=9, offset=3)
    b = oracle.verify_stage(zs, zl, tok, tau=0.3, mode=oracle.STRICT, seed=9, offset=3)
    assert np.array_equal(a["accept_len"], b["accept_len"]) and np.array_equal(a["next_token"], b["next_token"])
    # and with a threshold it accepts a superset of both rules
    c = oracle.verify_stage(zs, zl, tok, tau=0.05, mode=oracle.FUZZY_SD_FALLBACK, seed=9, offset=3)
    f = oracle.verify_stage(zs, zl, tok, tau=0.05, mode=oracle.FUZZY, seed=9, offset=3)
    assert np.array_equal(c["accept_bits"], np.maximum(b["accept_bits"], f["accept_bits"]))


def test_strict_accept_uses_ratio_of_token_probabilities(oracle):
    # p(x)/q(x) >= 1 -> always accepted; p(x) = 0 -> never accepted.
    zl = _logits_from_probs([0.7, 0.3, 0.0]).reshape(1, 1, 3)
    zs = _logits_from_probs([0.3, 0.3, 0.4]).reshape(1, 1, 3)
    for off in range(64):
        assert oracle.verify_stage(zs, zl, [[0]], 0, mode=oracle.STRICT, offset=off)["accept_len"][0] == 1
        assert oracle.verify_stage(zs, zl, [[1]], 0, mode=oracle.STRICT, offset=off)["accept_len"][0] == 1
        out = oracle.verify_stage(zs, zl, [[2]], 0, mode=oracle.STRICT, offset=off)
        assert out["accept_len"][0] == 0 and out["next_token"][0] == 0   # residual is (0.4, 0, 0)
    # ratio 0.5: accepted iff u < 0.5
    zl = _logits_from_probs([0.25, 0.75]).reshape(1, 1, 2)
    zs = _logits_from_probs([0.5, 0.5]).reshape(1, 1, 2)
    for off in range(200):
        u, _ = oracle.row_uniforms(0, off, 0)
        got = oracle.verify_stage(zs, zl, [[0]], 0, mode=oracle.STRICT, offset=off)["accept_len"][0]
        assert got == (1 if u < 0.5 else 0)


def test_flags_force_rejection(oracle):
    V = 8
    zl = np.zeros((1, 3, V))
    zs = np.zeros((1, 3, V))
    zs[0, 1, 3] = np.nan
    out = oracle.verify_stage(zs, zl, [[0, 0, 0]], tau=1.0)
    assert out["accept_len"][0] == 1 and out["next_token"][0] == -2
    assert out["row_flags"][0].tolist() == [0, oracle.FLAG_SMALL_NONFINITE, 0]
    zs[0, 1, 3] = 0.0
    zl[0, 0, 2] = np.inf
    out = oracle.verify_stage(zs, zl, [[0, 0, 0]], tau=1.0)
    assert out["accept_len"][0] == 0 and out["row_flags"][0, 0] == oracle.FLAG_LARGE_NONFINITE
    zl[0, 0, 2] = 0.5
    out = oracle.verify_stage(zs, zl, [[0, V, 0]], tau=1.0)   # out-of-range token at position 1
    assert out["accept_len"][0] == 1 and out["row_flags"][0, 1] == oracle.FLAG_TOKEN_RANGE
    assert out["next_token"][0] >= 0   # identical rows there: residual is zero, draw comes from p_large
    out = oracle.verify_stage(zs, zl, [[0, -1, 0]], tau=1.0)
    assert out["accept_len"][0] == 1


def test_n_valid_limits_the_scan(oracle):
    rng = np.random.default_rng(8)
    B, K, V = 4, 6, 20
    zl = rng.normal(0, 2, (B, K, V))
    tok = rng.integers(0, V, (B, K))
    out = oracle.verify_stage(zl, zl, tok, tau=0.0, n_valid=[0, 2, 6, 3])
    assert out["accept_len"].tolist() == [0, 2, 6, 3] and np.all(out["next_token"] == -1)


# ---------------------------------------------------------------- two-stage wrapper (Fig. 1)
def test_pyramid_composition(oracle):
    rng = np.random.default_rng(9)
    B, K_d, K_q, V = 10, 6, 4, 40
    zt_full = rng.normal(0, 3, (B, K_d, V)).astype(np.float32)
    zq = (zt_full + rng.normal(0, 0.7, (B, K_d, V))).astype(np.float32)
    zd = (zt_full + rng.normal(0, 1.5, (B, K_d, V))).astype(np.float32)
    zt = np.ascontiguousarray(zt_full[:, :K_q])
    tok = rng.integers(0, V, (B, K_d)).astype(np.int32)
    tau_q, tau_t, seed, off = 0.25, 0.1, 5, 40
    out = oracle.verify(zd, zq, zt, tok, tau_q, tau_t, seed=seed, offset=off)
    s1 = oracle.verify_stage(zd, zq, tok, tau_q, seed=seed, offset=off)
    assert np.array_equal(out["accept_len_q"], s1["accept_len"])
    assert np.array_equal(out["next_token_q"], s1["next_token"])
    seen_cut = seen_short = False
    for b in range(B):
        L1, t1 = s1["accept_len"][b], s1["next_token"][b]
        n2 = min(K_q, L1 + (1 if t1 >= 0 else 0))
        assert out["n_window"][b] == n2
        w = list(tok[b, :L1]) + ([t1] if t1 >= 0 else [])
        assert out["window"][b, :n2].tolist() == [int(x) for x in w[:n2]]
        seen_cut |= len(w) > K_q
        seen_short |= n2 < K_q
    assert seen_cut and seen_short
    s2 = oracle.verify_stage(np.ascontiguousarray(zq[:, :K_q]), zt, out["window"], tau_t, seed=seed,
                             offset=off + 1, n_valid=out["n_window"])
    assert np.array_equal(out["accept_len"], s2["accept_len"])
    assert np.array_equal(out["next_token"], s2["next_token"])
    assert np.all(out["accept_len"] <= out["n_window"])


def test_pyramid_all_accepted_first_stage(oracle):
    rng = np.random.default_rng(10)
    B, K_d, K_q, V = 3, 5, 3, 16
    z = rng.normal(0, 2, (B, K_d, V))
    tok = rng.integers(0, V, (B, K_d))
    out = oracle.verify(z, z, np.ascontiguousarray(z[:, :K_q]), tok, 0.0, 0.0)
    assert np.all(out["accept_len_q"] == K_d) and np.all(out["next_token_q"] == -1)
    assert np.all(out["n_window"] == K_q) and np.all(out["accept_len"] == K_q) and np.all(out["next_token"] == -1)
    assert np.array_equal(out["window"], tok[:, :K_q])


# ---------------------------------------------------------------- fused LM-head logits
def test_pyramid_assisted_qualifier_stage_keeps_the_fuzzy_target_stage(oracle):
    # Sec. 3.4 (PSD_A): assisted decoding takes the place of tau_Q only; the target stage keeps tau_T.
    # (a) composition on random inputs: stage 1 is the assisted stage, stage 2 the fuzzy stage on the window.
    rng = np.random.default_rng(19)
    B, K_d, K_q, V = 12, 5, 3, 30
    zt_full = rng.normal(0, 3, (B, K_d, V)).astype(np.float32)
    zq = (zt_full + rng.normal(0, 0.7, (B, K_d, V))).astype(np.float32)
    zd = (zt_full + rng.normal(0, 1.0, (B, K_d, V))).astype(np.float32)
    zt = np.ascontiguousarray(zt_full[:, :K_q])
    tok = np.stack([[rng.choice(V, p=sp_softmax(zd[b, k])) for k in range(K_d)] for b in range(B)]).astype(np.int32)
    out = oracle.verify(zd, zq, zt, tok, 0.9, 0.15, mode=oracle.ASSISTED, mode_t=oracle.FUZZY, seed=3, offset=20)
    s1 = oracle.verify_stage(zd, zq, tok, 0.9, mode=oracle.ASSISTED, seed=3, offset=20)
    assert np.array_equal(out["accept_len_q"], s1["accept_len"]) and np.array_equal(out["next_token_q"], s1["next_token"])
    assert 0 < s1["accept_len"].sum() < B * K_d            # tau_q = 0.9 > ln 2 would accept everything if it were used
    s2 = oracle.verify_stage(np.ascontiguousarray(zq[:, :K_q]), zt, out["window"], 0.15, mode=oracle.FUZZY, seed=3,
                             offset=21, n_valid=out["n_window"])
    assert np.array_equal(out["accept_len"], s2["accept_len"]) and np.array_equal(out["next_token"], s2["next_token"])
    same = oracle.verify(zd, zq, zt, tok, 0.9, 0.15, mode=oracle.ASSISTED, seed=3, offset=20)   # mode_t defaults to mode
    s2a = oracle.verify_stage(np.ascontiguousarray(zq[:, :K_q]), zt, out["window"], 0.15, mode=oracle.ASSISTED, seed=3,
                              offset=21, n_valid=out["n_window"])
    assert np.array_equal(same["accept_len"], s2a["accept_len"]) and not np.array_equal(same["accept_len"], out["accept_len"])
    # (b) the laws, K_d = K_q = 1, V = 16: the window token (draft token if accepted, else a draw from the
    # qualifier) follows min(p_q, p_d) + (1 - sum min) * p_q; a target stage with tau_T above ln 2 accepts it
    # whatever it is (threshold rule: the token plays no part), and with tau_T < 0 rejects it and draws from
    # the residual max(0, p_t - p_q), again whatever the window token was.
    V, n = 16, 300_000
    p_d, p_q, p_t = (sp_softmax(rng.normal(0, 1.5, V)) for _ in range(3))
    x = rng.choice(V, size=n, p=p_d).astype(np.int32).reshape(n, 1)
    zd1, zq1, zt1 = (np.broadcast_to(_logits_from_probs(p), (n, 1, V)).copy() for p in (p_d, p_q, p_t))
    acc_all = oracle.verify(zd1, zq1, zt1, x, 0.0, 1.0, mode=oracle.ASSISTED, mode_t=oracle.FUZZY, seed=4, offset=6, n_threads=8)
    assert np.all(acc_all["n_window"] == 1) and np.all(acc_all["accept_len"] == 1) and np.all(acc_all["next_token"] == -1)
    law = np.minimum(p_q, p_d) + (1 - np.minimum(p_q, p_d).sum()) * p_q
    counts = np.bincount(acc_all["window"][:, 0], minlength=V)
    assert stats.chisquare(counts, law * n).pvalue > 1e-3
    assert stats.chisquare(counts, p_q * n).pvalue < 1e-6 and stats.chisquare(counts, p_d * n).pvalue < 1e-6
    rej_all = oracle.verify(zd1, zq1, zt1, x, 0.0, -1.0, mode=oracle.ASSISTED, mode_t=oracle.FUZZY, seed=4, offset=6, n_threads=8)
    assert np.all(rej_all["accept_len"] == 0) and np.array_equal(rej_all["window"], acc_all["window"])
    resid = np.maximum(p_t - p_q, 0.0)
    live = resid > 0
    counts = np.bincount(rej_all["next_token"], minlength=V)
    assert np.all(counts[~live] == 0)
    assert stats.chisquare(counts[live], resid[live] / resid.sum() * n).pvalue > 1e-3


def test_lmhead_logits_match_library_matmul(oracle):
    import torch
    g = torch.Generator().manual_seed(0)
    h = torch.randn((5, 24), generator=g).to(torch.bfloat16)
    W = (torch.randn((24, 37), generator=g) * 0.02).to(torch.bfloat16)
    got = oracle.lmhead_logits(h.view(torch.int16).numpy().view(np.uint16), W.view(torch.int16).numpy().view(np.uint16))
    ref = h.double().numpy() @ W.double().numpy()
    np.testing.assert_allclose(got, ref, rtol=1e-13, atol=1e-15)


def test_mixed_stage_equals_plain_stage_on_same_values(oracle):
    import torch
    g = torch.Generator().manual_seed(1)
    zs = torch.randn((2, 3, 33), generator=g).mul(3).to(torch.bfloat16)
    zl = torch.randn((2, 3, 33), generator=g).mul(3).to(torch.bfloat16)
    tok = torch.randint(0, 33, (2, 3), generator=g).numpy()
    zs_b = zs.view(torch.int16).numpy().view(np.uint16)
    a = oracle.verify_stage_mixed(zs_b, zl.double().numpy(), tok, 0.3, seed=2, offset=9)
    b = oracle.verify_stage(zs.double().numpy(), zl.double().numpy(), tok, 0.3, seed=2, offset=9)
    assert np.array_equal(a["accept_len"], b["accept_len"]) and np.array_equal(a["next_token"], b["next_token"])
    np.testing.assert_array_equal(a["div"], b["div"])


def test_seq_ids_select_the_philox_rows_of_the_full_batch(oracle):
    rng = np.random.default_rng(12)
    B, K, V = 6, 3, 24
    zl = rng.normal(0, 2, (B, K, V))
    zs = zl + rng.normal(0, 1, (B, K, V))
    tok = rng.integers(0, V, (B, K))
    full = oracle.verify_stage(zs, zl, tok, 0.0, mode=oracle.STRICT, seed=4, offset=2)
    pick = [4, 1]
    part = oracle.verify_stage(zs[pick], zl[pick], tok[pick], 0.0, mode=oracle.STRICT, seed=4, offset=2, seq_ids=pick)
    assert np.array_equal(part["accept_len"], full["accept_len"][pick])
    assert np.array_equal(part["next_token"], full["next_token"][pick])


# ---------------------------------------------------------------- bonus token (all positions accepted)
def test_bonus_uniform_counter_layout(oracle):
    # counter = (b, 1, offset_lo, offset_hi): word 1 of the counter set apart from every row's (row, 0, ...)
    seed, offset, b = 0x1122334455667788, 0x99AABBCCDDEEFF00, 5
    w = oracle.philox4x32_10([b, 1, offset & 0xFFFFFFFF, offset >> 32], [seed & 0xFFFFFFFF, seed >> 32])
    assert oracle.bonus_uniform(seed, offset, b) == (int(w[1]) >> 8) / 2.0**24
    assert oracle.bonus_uniform(seed, offset, b) != oracle.row_uniforms(seed, offset, b)[1]


def _accepting_case(rng, B, K, V):
    """Identical small and large rows (divergence exactly 0: fuzzy tau = 0 accepts) + a free bonus row."""
    zs = rng.normal(size=(B, K, V)).astype(np.float32)
    zl = np.concatenate([zs, rng.normal(size=(B, 1, V)).astype(np.float32)], axis=1)
    tok = rng.integers(0, V, size=(B, K)).astype(np.int32)
    return zs, zl, tok


def test_bonus_token_is_the_hot_index_of_the_row_after_the_window(oracle):
    rng = np.random.default_rng(5)
    B, K, V = 4, 3, 9
    zs, zl, tok = _accepting_case(rng, B, K, V)
    for j in range(K + 1):                       # row j of the large model: one-hot at index j + 2
        zl[:, j, :] = -np.inf
        zl[:, j, j + 2] = 1.5
    zs[:] = zl[:, :K]
    nv = np.array([0, 1, 2, 3], np.int32)        # the bonus row is the one after the last valid position
    for offset in range(5):
        out = oracle.verify_stage_bonus(zs, zl, tok, 0.0, oracle.FUZZY, 3, offset, n_valid=nv)
        assert np.array_equal(out["accept_len"], nv)
        assert np.array_equal(out["next_token"], nv + 2)


def test_bonus_row_is_ignored_when_a_position_is_rejected(oracle):
    rng = np.random.default_rng(6)
    B, K, V = 6, 4, 12
    zs = rng.normal(size=(B, K, V)).astype(np.float32)
    zl = rng.normal(size=(B, K + 1, V)).astype(np.float32)
    tok = rng.integers(0, V, size=(B, K)).astype(np.int32)
    plain = oracle.verify_stage(zs, np.ascontiguousarray(zl[:, :K]), tok, 0.02, oracle.FUZZY, 1, 2)
    bonus = oracle.verify_stage_bonus(zs, zl, tok, 0.02, oracle.FUZZY, 1, 2)
    assert np.all(plain["accept_len"] < K)       # random rows: every sequence has a rejection
    assert np.array_equal(plain["accept_len"], bonus["accept_len"])
    assert np.array_equal(plain["next_token"], bonus["next_token"])


def test_bonus_tokens_follow_the_large_models_distribution(oracle):
    rng = np.random.default_rng(7)
    B, K, V = 30000, 1, 16
    row = rng.normal(size=V).astype(np.float32)
    bon = (2.0 * rng.normal(size=V)).astype(np.float32)
    zs = np.broadcast_to(row, (B, K, V)).copy()
    zl = np.concatenate([zs, np.broadcast_to(bon, (B, 1, V))], axis=1).copy()
    tok = np.zeros((B, K), np.int32)
    out = oracle.verify_stage_bonus(zs, zl, tok, 0.0, oracle.FUZZY, 11, 4, n_threads=4)
    assert np.all(out["accept_len"] == 1)
    counts = np.bincount(out["next_token"], minlength=V)
    p = sp_softmax(bon.astype(np.float64))
    assert stats.chisquare(counts, p * B).pvalue > 1e-3
    assert stats.chisquare(counts, sp_softmax(row.astype(np.float64)) * B).pvalue < 1e-6   # not the scoring row's law


def test_bonus_row_without_a_distribution_gives_the_invalid_marker(oracle):
    rng = np.random.default_rng(8)
    zs, zl, tok = _accepting_case(rng, 3, 2, 8)
    zl[0, 2, 3] = np.nan
    zl[1, 2, :] = -np.inf
    out = oracle.verify_stage_bonus(zs, zl, tok, 0.0, oracle.FUZZY, 0, 0)
    assert np.array_equal(out["accept_len"], [2, 2, 2])
    assert out["next_token"][0] == -2 and out["next_token"][1] == -2 and 0 <= out["next_token"][2] < 8


def test_pyramid_bonus_composition(oracle):
    """Two stages with a K_q+1-row target: stage 1, the window and the accept lengths are those of the plain
    pyramid; only fully accepted windows get a token, drawn from the target's row after the window."""
    rng = np.random.default_rng(9)
    B, K_d, K_q, V = 8, 4, 2, 10
    zq = rng.normal(size=(B, K_d, V)).astype(np.float32)
    zd = zq.copy()                                   # draft == qualifier: stage 1 accepts everything
    zt = np.concatenate([zq[:, :K_q], np.full((B, 1, V), -np.inf, np.float32)], axis=1)
    zt[:, K_q, 7] = 0.0                              # bonus row: one-hot at 7
    zt[B // 2:, 1] = rng.normal(size=(B - B // 2, V)) * 3   # second half: target disagrees at position 1
    tok = rng.integers(0, V, size=(B, K_d)).astype(np.int32)
    plain = oracle.verify(zd, zq, np.ascontiguousarray(zt[:, :K_q]), tok, 0.0, 0.0, oracle.FUZZY, 2, 6)
    out = oracle.verify_bonus(zd, zq, zt, tok, 0.0, 0.0, oracle.FUZZY, 2, 6)
    assert np.array_equal(out["accept_len_q"], np.full(B, K_d)) and np.array_equal(out["accept_len"], plain["accept_len"])
    assert np.all(out["accept_len"][:B // 2] == K_q) and np.all(out["next_token"][:B // 2] == 7)
    assert np.all(out["accept_len"][B // 2:] == 1)
    assert np.array_equal(out["next_token"][B // 2:], plain["next_token"][B // 2:])
