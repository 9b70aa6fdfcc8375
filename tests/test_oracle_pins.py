"""Pins for the oracle's arithmetic against what the paper and the mathematics fix.

Each test states the passage it leans on.  None of them re-types the oracle's own
formula path: the distributions are rebuilt here from scipy's softmax, laws are counted
by bisection over the uniform lattice, and whole rows are enumerated by brute force.
"""
import itertools
import math

import numpy as np
import pytest
from scipy.special import softmax as sp_softmax
from scipy.stats import chi2 as chi2_dist

from oracle import cos_oracle as orc

WE, LL = orc.COMBINE_PROB_ENSEMBLE, orc.COMBINE_LOGIT_LINEAR
LATTICE = 1 << 23            # u takes the values (2m+1) * 2^-24, m = 0 .. 2^23 - 1


def lattice_u(m):
    return (2 * m + 1) * 2.0 ** -24


def rng_logits(seed, n, V, scale=2.0):
    g = np.random.default_rng(seed)
    return g.normal(size=(n, V)) * scale


def cfg_we(n, V, w, T=1.0, gamma=1):
    return orc.OracleConfig(n=n, combine=WE, weights=w, temperature=T, gamma=gamma, vocab=V)


def cfg_ll(n, V, w, T=1.0, gamma=1, mask_model=-1, alpha=1.0):
    return orc.OracleConfig(n=n, combine=LL, weights=w, temperature=T, gamma=gamma, vocab=V,
                            mask_model=mask_model, mask_alpha=alpha)


# --------------------------------------------------------------------------------------
# distributions: special cases that reduce to a library softmax
# --------------------------------------------------------------------------------------
@pytest.mark.parametrize("T", [1.0, 0.7, 2.5])
def test_weighted_ensemble_is_convex_mix_of_library_softmaxes(T):
    """Eq. 4 with each distribution a tempered softmax."""
    V = 50
    l = rng_logits(1, 3, V)
    w = np.array([0.5, 0.3, 0.2], dtype=np.float32)
    Tf = float(np.float32(T))
    r, q, ok = orc.position_distributions(l, cfg_we(3, V, w, T), proposer=1)
    ref = sum(float(w[i]) * sp_softmax(l[i] / Tf) for i in range(3))
    assert ok
    np.testing.assert_allclose(r, ref, rtol=1e-13, atol=0)
    np.testing.assert_allclose(q, sp_softmax(l[1] / Tf), rtol=1e-13)
    assert abs(r.sum() - float(w.astype(np.float64).sum())) < 1e-12   # fp32 weights sum to 1 only to ~1e-8


def test_single_model_and_one_hot_weights_reduce_to_softmax():
    V = 33
    l = rng_logits(2, 3, V)
    r, q, _ = orc.position_distributions(l[:1], cfg_we(1, V, [1.0]), 0)
    np.testing.assert_allclose(r, sp_softmax(l[0]), rtol=1e-13)
    np.testing.assert_array_equal(r, q)
    r, _, _ = orc.position_distributions(l, cfg_we(3, V, [0.0, 0.0, 1.0]), 0)
    np.testing.assert_allclose(r, sp_softmax(l[2]), rtol=1e-13)
    r, _, _ = orc.position_distributions(l, cfg_ll(3, V, [0.0, 1.0, 0.0]), 0)
    np.testing.assert_allclose(r, sp_softmax(l[1]), rtol=1e-13)


@pytest.mark.parametrize("mu,T", [(0.1, 1.0), (0.5, 1.0), (0.5, 0.6)])
def test_contrastive_is_softmax_of_logit_difference(mu, T):
    """Eq. 5: r = Softmax(l^p - mu l^q), here with the expert stored as model 0."""
    V = 40
    l = rng_logits(3, 2, V, scale=3.0)
    muf, Tf = float(np.float32(mu)), float(np.float32(T))
    r, q, _ = orc.position_distributions(l, cfg_ll(2, V, [1.0, -mu], T), proposer=1)
    np.testing.assert_allclose(r, sp_softmax((l[0] - muf * l[1]) / Tf), rtol=1e-12)
    np.testing.assert_allclose(q, sp_softmax(l[1] / Tf), rtol=1e-13)


def test_plausibility_mask_properties():
    V = 200
    l = rng_logits(4, 2, V, scale=3.0)
    alpha = 0.1
    cfg = cfg_ll(2, V, [1.0, -0.5], T=1.0, mask_model=0, alpha=alpha)
    r, _, ok = orc.position_distributions(l, cfg, proposer=1)
    p_e = sp_softmax(l[0])
    keep = p_e >= float(np.float32(alpha)) * p_e.max() * (1 - 1e-12)
    assert ok and abs(r.sum() - 1.0) < 1e-12
    assert np.all(r[~keep] == 0.0) and np.all(r[keep] > 0.0)
    assert 1 < keep.sum() < V                                   # the case is not degenerate
    # on the kept set r is the renormalised unmasked contrastive softmax
    full = sp_softmax(l[0] - 0.5 * l[1])
    np.testing.assert_allclose(r[keep], full[keep] / full[keep].sum(), rtol=1e-12)
    # a vanishing threshold keeps everything: plain Eq. 5 again
    r_all, _, _ = orc.position_distributions(l, cfg_ll(2, V, [1.0, -0.5], T=1.0, mask_model=0, alpha=1e-30), 1)
    np.testing.assert_allclose(r_all, full, rtol=1e-12)


def test_ensemble_config_validation():
    with pytest.raises(ValueError):
        cfg_we(2, 8, [0.7, 0.7])
    with pytest.raises(ValueError):
        cfg_we(2, 8, [1.5, -0.5])
    with pytest.raises(ValueError):
        orc.OracleConfig(n=2, combine=WE, weights=[0.5, 0.5], temperature=1.0, gamma=1, vocab=8, mask_model=0)
    cfg_ll(2, 8, [1.5, -0.5])                                    # negative weights are fine at logit level


def test_bf16_and_f32_upcasts_are_exact():
    bits = np.array([0x3F80, 0xBF80, 0x4049, 0x0000, 0x8000, 0x7F80, 0xFF80, 0x0001], dtype=np.uint16)
    v = orc.to_float64(bits, "bf16")
    assert v[0] == 1.0 and v[1] == -1.0 and v[2] == 3.140625 and v[3] == 0.0
    assert np.isposinf(v[5]) and np.isneginf(v[6]) and v[7] == 2.0 ** -133
    f = np.array([0.1, 1e-20, 3.5], dtype=np.float32)
    assert np.array_equal(orc.to_float64(f, "f32"), f.astype(np.float64))
    # IEEE half, decoded here from the bit fields (1 sign, 5 exponent, 10 fraction bits)
    hb = np.array([0x3C00, 0xC000, 0x3555, 0x0001, 0x03FF, 0x7BFF, 0x7C00, 0xFC00, 0x8000], dtype=np.uint16)
    want = []
    for x in hb.tolist():
        sgn, ex, fr = -1.0 if x >> 15 else 1.0, (x >> 10) & 31, x & 1023
        want.append(sgn * (math.inf if ex == 31 else (fr * 2.0 ** -24 if ex == 0 else (1 + fr / 1024) * 2.0 ** (ex - 15))))
    got = orc.to_float64(hb.view(np.float16), "f16")
    assert np.array_equal(got, np.array(want)) and np.signbit(got[8])


# --------------------------------------------------------------------------------------
# ratio test: invariants of Sec. 3.2
# --------------------------------------------------------------------------------------
def test_ratio_never_below_proposer_weight():
    """Thm 3.2: min(1, r/q) >= lambda for the ensemble, at every token."""
    V = 64
    w = np.array([0.4, 0.3, 0.2, 0.1], dtype=np.float32)
    for seed in range(5):
        l = rng_logits(10 + seed, 4, V, scale=4.0)
        for pi in range(4):
            cfg = cfg_we(4, V, w)
            for d in range(V):
                res = orc.verify_position(l, cfg, pi, d, 0.5, 0.5)
                assert res.ratio >= float(w[pi]) * (1 - 1e-12)


def test_proposer_equal_to_target_accepts_everything():
    """Eq. 4 with lambda = 1: r = q, ratio 1, every draft accepted, bonus emitted."""
    n, B, g, V = 2, 7, 5, 30
    gen = np.random.default_rng(5)
    logits = gen.normal(size=(n, B, g + 1, V)).astype(np.float32)
    drafts = gen.integers(0, V, size=(B, g))
    cfg = cfg_we(n, V, [1.0, 0.0], gamma=g)
    out = orc.verify(logits, "f32", drafts, np.zeros(B, int), cfg, seed=99, offset=3)
    assert np.all(out["accept_count"] == g)
    assert np.array_equal(out["out_tokens"][:, :g], drafts)
    assert np.all(out["out_tokens"][:, g] >= 0)
    assert np.all(out["ratio"][:, :g] == 1.0)
    assert np.all(out["row_status"] == 0)


def test_accept_decision_is_u_le_min_one_ratio_including_equality():
    V = 4
    l = np.log(np.array([[0.5, 0.25, 0.125, 0.125], [0.125, 0.125, 0.25, 0.5]]))
    cfg = cfg_we(2, V, [0.5, 0.5])
    # proposer 0, draft 0: r = 0.3125, q = 0.5, ratio 0.625 (a dyadic number: representable u)
    res = orc.verify_position(l, cfg, 0, 0, 0.625, 0.5)
    assert abs(res.ratio - 0.625) < 1e-15
    thr = res.ratio
    assert orc.verify_position(l, cfg, 0, 0, thr, 0.5).accept            # equality accepts ("<=")
    assert not orc.verify_position(l, cfg, 0, 0, np.nextafter(thr, 1.0), 0.5).accept
    assert orc.verify_position(l, cfg, 0, 0, np.nextafter(thr, 0.0), 0.5).accept
    # ratio > 1 (draft 3 is under-proposed): accepted for every u < 1
    assert orc.verify_position(l, cfg, 0, 3, 1.0 - 2.0 ** -24, 0.5).accept


def test_lambda_zero_is_textbook_speculative_decoding():
    """Sec. 3.2 (quality-speed trade-off): with weight 0 on the proposer the target is the
    other model alone, i.e. Eq. 2 and the residual norm(max(0, p - q))."""
    V = 12
    l = rng_logits(21, 2, V)
    p, q = sp_softmax(l[1]), sp_softmax(l[0])
    cfg = cfg_we(2, V, [0.0, 1.0])
    resid = np.maximum(p - q, 0)
    cdf = np.cumsum(resid) / resid.sum()
    for d in range(V):
        for u in (0.03, 0.41, 0.77, 0.999):
            res = orc.verify_position(l, cfg, 0, d, u, u)
            assert res.accept == (u <= min(1.0, p[d] / q[d]))
            assert res.cand == int(np.searchsorted(cdf, u, side="left"))


# --------------------------------------------------------------------------------------
# exact output law on small vocabularies (App. A.1), by counting lattice uniforms
# --------------------------------------------------------------------------------------
def _count_accepting_u(l, cfg, pi, d, dist):
    """Number of lattice values of u_acc for which draft d is accepted.  The decision is
    monotone in u, so bisection over the lattice index counts it exactly."""
    if not orc.verify_position(l, cfg, pi, d, lattice_u(0), 0.5, dist=dist).accept:
        return 0
    lo, hi = 0, LATTICE - 1                      # lo accepted; find the last accepted index
    if orc.verify_position(l, cfg, pi, d, lattice_u(hi), 0.5, dist=dist).accept:
        return LATTICE
    while hi - lo > 1:
        mid = (lo + hi) // 2
        if orc.verify_position(l, cfg, pi, d, lattice_u(mid), 0.5, dist=dist).accept:
            lo = mid
        else:
            hi = mid
    return lo + 1


def _count_sampled_u(l, cfg, pi, d, V, dist):
    """For a rejected draft (u_acc = 1 - 2^-24 rejects whenever ratio < 1) or the bonus
    (d None): how many lattice values of u_smp map to each token.  cand is non-decreasing
    in u, so each token's block is found by bisection."""
    def cand(m):
        return orc.verify_position(l, cfg, pi, d, 1.0 - 2.0 ** -24, lattice_u(m), dist=dist).cand
    counts = np.zeros(V, dtype=np.int64)
    start = 0
    while start < LATTICE:
        k = cand(start)
        lo, hi = start, LATTICE - 1              # find the last m with cand(m) == k
        if cand(hi) == k:
            end = hi
        else:
            while hi - lo > 1:
                mid = (lo + hi) // 2
                if cand(mid) <= k:
                    lo = mid
                else:
                    hi = mid
            end = lo
        counts[k] += end - start + 1
        start = end + 1
    return counts


LAW_CASES = [
    ("we2", lambda V: cfg_we(2, V, [0.5, 0.5]), 2, 0),
    ("we3_T", lambda V: cfg_we(3, V, [0.2, 0.5, 0.3], T=0.7), 3, 1),
    ("cd", lambda V: cfg_ll(2, V, [1.0, -0.5]), 2, 1),
    ("cd_mask", lambda V: cfg_ll(2, V, [1.0, -0.5], mask_model=0, alpha=0.1), 2, 1),
    ("realign", lambda V: cfg_ll(2, V, [1.5, -0.5], T=1.3), 2, 0),
]


@pytest.mark.parametrize("name,mk,n,pi", LAW_CASES, ids=[c[0] for c in LAW_CASES])
@pytest.mark.parametrize("V", [3, 8])
def test_output_token_law_equals_combined_distribution(name, mk, n, pi, V):
    """App. A.1: P(x = x') = q(x') min(1, r/q) + P(reject) * res(x')/S = r(x').

    q is the law the drafts are drawn from; the accept probability and the resample law
    are counted over all 2^23 values the uniforms can take."""
    l = rng_logits(100 + V, n, V, scale=1.5)
    cfg = mk(V)
    dist = orc.position_distributions(l, cfg, pi)
    # independent statement of the target and proposal laws
    Tf = cfg.temperature
    q_ref = sp_softmax(l[pi] / Tf)
    if cfg.combine == WE:
        r_ref = sum(cfg.w64[i] * sp_softmax(l[i] / Tf) for i in range(n))
    else:
        c = sum(cfg.w64[i] * l[i] for i in range(n)) / Tf
        if cfg.mask_model >= 0:
            pe = sp_softmax(l[cfg.mask_model])
            c = np.where(pe >= cfg.mask_alpha * pe.max(), c, -np.inf)
        r_ref = sp_softmax(c)
    p_acc = np.array([_count_accepting_u(l, cfg, pi, d, dist) for d in range(V)]) / LATTICE
    np.testing.assert_allclose(p_acc, np.minimum(1.0, r_ref / q_ref), atol=2.0 ** -22)
    p_reject = float(np.sum(q_ref * (1.0 - p_acc)))
    # P(reject) = sum max(r - q, 0) = 1/2 sum |r - q|   (App. A.1; Eq. 7)
    assert abs(p_reject - np.maximum(r_ref - q_ref, 0).sum()) < 1e-5
    assert abs(p_reject - 0.5 * np.abs(r_ref - q_ref).sum()) < 1e-5
    some_rejectable = next(d for d in range(V) if r_ref[d] < q_ref[d])
    counts = _count_sampled_u(l, cfg, pi, some_rejectable, V, dist)
    p_res = counts / LATTICE
    resid = np.maximum(r_ref - q_ref, 0)
    assert np.all(np.abs(counts - resid / resid.sum() * LATTICE) <= 1.0 + 1e-6)
    law = q_ref * p_acc + p_reject * p_res
    np.testing.assert_allclose(law, r_ref, atol=1e-6)
    # the bonus sample follows r itself (gamma = 0 is direct sampling from r)
    counts_b = _count_sampled_u(l, cfg, pi, None, V, dist)
    assert np.all(np.abs(counts_b - r_ref * LATTICE) <= 1.0 + 1e-6)


def test_residual_mass_identity_in_the_oracle():
    """sum max(0, r - q) computed by the oracle equals 1/2 sum |r - q| and 1 - alpha (Eq. 7)."""
    V = 300
    l = rng_logits(31, 2, V, scale=3.0)
    cfg = cfg_we(2, V, [0.5, 0.5])
    r, q, _ = orc.position_distributions(l, cfg, 0)
    res = orc.verify_position(l, cfg, 0, 5, 0.5, 0.5)
    assert abs(res.S - 0.5 * np.abs(sp_softmax(l[0]) * 0.5 - sp_softmax(l[1]) * 0.5).sum()) < 1e-12
    assert abs((1.0 - res.S) - orc.acceptance_rate(r, q)) < 1e-12


def test_gamma_zero_is_direct_sampling_from_r():
    n, B, V = 2, 40, 17
    gen = np.random.default_rng(8)
    logits = gen.normal(size=(n, B, 1, V)).astype(np.float32) * 2
    cfg = cfg_ll(2, V, [1.5, -0.5], gamma=0)
    out = orc.verify(logits, "f32", np.zeros((B, 0), int), np.zeros(B, int), cfg, seed=4, offset=0)
    _, us = orc.position_uniforms(4, 0, B, 1)
    for b in range(B):
        l = logits[:, b, 0, :].astype(np.float64)
        r = sp_softmax(1.5 * l[0] - 0.5 * l[1])
        k = int(np.searchsorted(np.cumsum(r), us[b, 0] * np.cumsum(r)[-1], side="left"))
        assert out["accept_count"][b] == 0 and out["out_tokens"][b, 0] == k


def test_inverse_cdf_conventions():
    mass = np.array([0.0, 0.25, 0.0, 0.5, 0.25, 0.0])
    assert orc.inverse_cdf(mass, 2.0 ** -24)[0] == 1            # zero-mass head is never returned
    assert orc.inverse_cdf(mass, 0.25)[0] == 1                  # CDF_k >= u*S with equality: smallest k
    assert orc.inverse_cdf(mass, np.nextafter(0.25, 1))[0] == 3
    assert orc.inverse_cdf(mass, 0.75)[0] == 3
    assert orc.inverse_cdf(mass, 1 - 2.0 ** -24)[0] == 4        # zero-mass tail is never returned
    k, total, lo, hi = orc.inverse_cdf(mass * 8, 0.5)
    assert (k, total, lo, hi) == (3, 8.0, 0.25, 0.75)           # unnormalised mass, normalised edges


# --------------------------------------------------------------------------------------
# whole-row semantics by brute force (Sec. 3.1: first rejection discards the tail)
# --------------------------------------------------------------------------------------
def test_row_law_by_enumeration_gamma2():
    """Enumerate every draft pair and a grid of uniforms at V = 3, gamma = 2 and compare the
    law of (accept_count, out_tokens) with the product form
      P(a=0,[t]) = res_0(t);  P(a=1,[d0,t]) = min(q_0,r_0)(d0) res_1(t);
      P(a=2,[d0,d1,t]) = min(q_0,r_0)(d0) min(q_1,r_1)(d1) r_2(t),
    res_j = max(r_j - q_j, 0) unnormalised."""
    n, g, V, G = 2, 2, 3, 24
    gen = np.random.default_rng(77)
    logits = gen.normal(size=(n, 1, g + 1, V)) * 1.2
    cfg = cfg_we(n, V, [0.5, 0.5], gamma=g)
    q = [sp_softmax(logits[0, 0, j]) for j in range(g + 1)]
    r = [0.5 * sp_softmax(logits[0, 0, j]) + 0.5 * sp_softmax(logits[1, 0, j]) for j in range(g + 1)]
    grid = (np.arange(G) + 0.5) / G
    law = {}
    for d0, d1 in itertools.product(range(V), repeat=2):
        pd = q[0][d0] * q[1][d1]
        # u_smp matters only at the emitting position, so one shared grid value is enough
        for ua0, ua1, us in itertools.product(grid, repeat=3):
            out = orc.verify(logits, "f64", [[d0, d1]], [0], cfg, 0, 0,
                             uniforms=([[ua0, ua1, 0.5]], [[us, us, us]]))
            key = (int(out["accept_count"][0]), tuple(int(t) for t in out["out_tokens"][0]))
            law[key] = law.get(key, 0.0) + pd / G ** 3
    tol = 3.0 / G
    seen = 0.0
    for (a, toks), prob in law.items():
        assert all(t == -1 for t in toks[a + 1:]) and all(t >= 0 for t in toks[: a + 1])
        # the drafts that do not appear in the key (rejected ones) are summed over inside `law`
        if a == 0:
            expect = np.maximum(r[0] - q[0], 0)[toks[0]]
        elif a == 1:
            expect = min(q[0][toks[0]], r[0][toks[0]]) * np.maximum(r[1] - q[1], 0)[toks[1]]
        else:
            expect = min(q[0][toks[0]], r[0][toks[0]]) * min(q[1][toks[1]], r[1][toks[1]]) * r[2][toks[2]]
        assert abs(prob - expect) < tol, (a, toks, prob, expect)
        seen += prob
    assert abs(seen - 1.0) < 1e-9


def test_first_rejection_discards_tail_and_status_scope():
    n, g, V = 2, 3, 5
    logits = np.zeros((n, 1, g + 1, V))
    logits[0, 0, :, 0] = 5.0          # proposer loves token 0
    logits[1, 0, :, 1] = 5.0          # the other model loves token 1
    logits[0, 0, 3, 2] = np.nan       # a non-finite position AFTER the first rejection
    cfg = cfg_we(n, V, [0.5, 0.5], gamma=g)
    ua = [[0.1, 0.99, 0.1, 0.5]]      # position 1 rejects (ratio ~0.5 < 0.99)
    out = orc.verify(logits, "f64", [[0, 0, 0]], [0], cfg, 0, 0, uniforms=(ua, [[0.5] * 4]))
    assert out["accept_count"][0] == 1
    assert out["out_tokens"][0, 0] == 0 and out["out_tokens"][0, 1] == 1     # residual mass sits on token 1
    assert list(out["out_tokens"][0, 2:]) == [-1, -1]
    assert out["row_status"][0] == 0                                           # discarded positions do not report
    # the same non-finite value before the rejection does report and stops the row there
    logits[0, 0, 0, 2] = np.inf
    out = orc.verify(logits, "f64", [[0, 0, 0]], [0], cfg, 0, 0, uniforms=(ua, [[0.5] * 4]))
    assert out["accept_count"][0] == 0 and out["out_tokens"][0, 0] == -1
    assert out["row_status"][0] & orc.STATUS_NONFINITE


def test_bad_draft_and_minus_inf_logits():
    n, g, V = 2, 1, 6
    gen = np.random.default_rng(3)
    logits = gen.normal(size=(n, 1, g + 1, V))
    logits[1, 0, 0, 4] = -np.inf                                # a token one model rules out is fine
    cfg = cfg_we(n, V, [0.5, 0.5], gamma=g)
    out = orc.verify(logits, "f64", [[V]], [0], cfg, 1, 1)      # draft outside the vocabulary
    assert out["accept_count"][0] == 0 and out["row_status"][0] == orc.STATUS_BAD_DRAFT
    assert 0 <= out["out_tokens"][0, 0] < V
    out = orc.verify(logits, "f64", [[-1]], [0], cfg, 1, 1)
    assert out["row_status"][0] == orc.STATUS_BAD_DRAFT
    out = orc.verify(logits, "f64", [[2]], [0], cfg, 1, 1)
    assert out["row_status"][0] == 0


# --------------------------------------------------------------------------------------
# statistics: chi-squared on the emitted token, expected accepted length
# --------------------------------------------------------------------------------------
def test_chi_squared_first_emitted_token_follows_r():
    """V = 64, 1e6 trials: drafts are drawn from q with numpy's own generator, the oracle
    decides with its Philox uniforms; the first emitted token must follow r (App. A.1)."""
    V, N = 64, 1_000_000
    l = rng_logits(64, 2, V, scale=1.5)
    cfg = cfg_we(2, V, [0.5, 0.5], gamma=1)
    dist = orc.position_distributions(l, cfg, 0)
    q_ref = sp_softmax(l[0])
    r_ref = 0.5 * sp_softmax(l[0]) + 0.5 * sp_softmax(l[1])
    drafts = np.random.default_rng(2024).choice(V, size=N, p=q_ref)
    ua, us = orc.position_uniforms(0xC0FFEE, 0, N, 1)
    counts = np.zeros(V, dtype=np.int64)
    accepted = 0
    for t in range(N):
        res = orc.verify_position(l, cfg, 0, int(drafts[t]), ua[t, 0], us[t, 0], dist=dist)
        counts[drafts[t] if res.accept else res.cand] += 1
        accepted += res.accept
    expected = r_ref * N
    stat = float(np.sum((counts - expected) ** 2 / expected))
    assert stat < chi2_dist.ppf(1 - 1e-6, V - 1), stat          # 63 d.o.f.
    alpha = 1.0 - 0.5 * np.abs(q_ref - r_ref).sum()              # Eq. 7
    assert abs(accepted / N - alpha) < 5 * math.sqrt(alpha * (1 - alpha) / N)


def test_expected_accepted_length_matches_closed_form():
    """App. A.2: with the same alpha at every position E[#accepted drafts] =
    sum_{k=1..gamma} alpha^k, and E[#tokens without bonus] = (1 - alpha^gamma)/(1 - alpha)."""
    n, B, g, V = 2, 20000, 4, 16
    l = rng_logits(5, n, V, scale=1.0)
    q_ref = sp_softmax(l[0])
    r_ref = 0.5 * q_ref + 0.5 * sp_softmax(l[1])
    alpha = 1.0 - 0.5 * np.abs(q_ref - r_ref).sum()
    logits = np.broadcast_to(l[:, None, None, :], (n, B, g + 1, V))
    drafts = np.random.default_rng(11).choice(V, size=(B, g), p=q_ref)
    cfg = cfg_we(n, V, [0.5, 0.5], gamma=g)
    out = orc.verify(logits, "f64", drafts, np.zeros(B, int), cfg, seed=77, offset=5)
    mean_acc = out["accept_count"].mean()
    expect = sum(alpha ** k for k in range(1, g + 1))
    # tokens per cycle when the bonus is not counted: min(accepted + 1, gamma)
    tokens_no_bonus = np.minimum(out["accept_count"] + 1, g).mean()
    assert abs(tokens_no_bonus - (1 - alpha ** g) / (1 - alpha)) < 0.03
    assert abs(mean_acc - expect) < 0.03
    assert np.all(out["row_status"] == 0)


def test_acceptance_falls_as_mu_grows():
    """Sec. 4.3: a larger contrastive coefficient moves r away from the proposer."""
    V = 500
    gen = np.random.default_rng(13)
    z = gen.normal(size=V)
    l = np.stack([3 * (0.8 * z + 0.6 * gen.normal(size=V)), 3 * (0.8 * z + 0.6 * gen.normal(size=V))])
    alphas = []
    for mu in (0.1, 0.2, 0.3, 0.4, 0.5):
        r, q, _ = orc.position_distributions(l, cfg_ll(2, V, [1.0, -mu]), proposer=0)
        alphas.append(orc.acceptance_rate(r, q))
    assert all(a > b for a, b in zip(alphas, alphas[1:]))


# --------------------------------------------------------------------------------------
# greedy mode (Sec. 4.1: T = 0 gives one-hot distributions)
# --------------------------------------------------------------------------------------
def test_greedy_is_the_zero_temperature_limit_and_breaks_ties_low():
    V = 20
    l = rng_logits(17, 2, V, scale=2.0)
    for mk in (lambda T: cfg_ll(2, V, [1.5, -0.5], T=T),
               lambda T: cfg_ll(2, V, [1.0, -0.5], T=T, mask_model=0, alpha=0.1)):
        r0, q0, ok = orc.position_distributions(l, mk(0.0), 1)
        rT, qT, _ = orc.position_distributions(l, mk(1e-3), 1)
        assert ok and r0.sum() == 1.0 and q0.sum() == 1.0 and set(np.unique(r0)) == {0.0, 1.0}
        assert np.argmax(rT) == np.argmax(r0) and rT.max() > 0.999
        assert np.argmax(qT) == np.argmax(q0)
    # ties: lowest index wins, for q, for the ensemble atoms and for the combined logits
    t = np.zeros((2, 6))
    t[0, [2, 4]] = 1.0
    t[1, [3, 5]] = 2.0
    r, q, _ = orc.position_distributions(t, cfg_we(2, 6, [0.25, 0.75], T=0.0), 0)
    assert q[2] == 1.0 and r[2] == 0.25 and r[3] == 0.75 and r.sum() == 1.0
    r, _, _ = orc.position_distributions(t, cfg_ll(2, 6, [1.0, 0.5], T=0.0), 0)   # c = [0,0,1,1,1,1]
    assert r[2] == 1.0


def test_greedy_verification_is_deterministic_argmax_comparison():
    n, B, g, V = 2, 30, 3, 25
    gen = np.random.default_rng(19)
    logits = (gen.normal(size=(n, B, g + 1, V)) * 2).astype(np.float32)
    cfg = cfg_ll(n, V, [1.5, -0.5], T=0.0, gamma=g)
    drafts = np.argmax(logits[0], axis=-1)[:, :g]                 # greedy proposer = model 0
    target = np.argmax(1.5 * logits[0].astype(np.float64) - 0.5 * logits[1].astype(np.float64), axis=-1)
    a = orc.verify(logits, "f32", drafts, np.zeros(B, int), cfg, seed=1, offset=0)
    b = orc.verify(logits, "f32", drafts, np.zeros(B, int), cfg, seed=999, offset=12345)
    assert np.array_equal(a["out_tokens"], b["out_tokens"])       # no dependence on the uniforms
    for row in range(B):
        k = 0
        while k < g and drafts[row, k] == target[row, k]:
            k += 1
        assert a["accept_count"][row] == k
        assert a["out_tokens"][row, k] == target[row, k]
    assert 0 < a["accept_count"].mean() < g                       # both outcomes occur


# --------------------------------------------------------------------------------------
# alternate proposals (Sec. 3.3, Algorithm 2): bonus token from a named model, proposer per position
# --------------------------------------------------------------------------------------
@pytest.mark.parametrize("name,mk,n,pi", LAW_CASES, ids=[c[0] for c in LAW_CASES])
@pytest.mark.parametrize("T0", [False, True])
def test_named_bonus_model_draws_from_that_models_own_law(name, mk, n, pi, T0):
    """Sec. 3.3: the token after gamma acceptances "is drawn from p" of the verifier, not from the
    combined law; Algorithm 2's Score returns it with its probability.  Counted over the uniform lattice
    against scipy's softmax of that model alone; at T = 0 it is that model's lowest-index argmax."""
    V = 8
    l = rng_logits(300 + n, n, V, scale=1.5)
    base = mk(V)
    for m in range(n):
        cfg = orc.OracleConfig(n=n, combine=base.combine, weights=list(base.w64), gamma=1, vocab=V,
                               temperature=0.0 if T0 else base.temperature, mask_model=base.mask_model,
                               mask_alpha=base.mask_alpha, bonus_model=m)
        if T0:
            res = orc.verify_position(l, cfg, pi, None, 0.3, 0.77)
            assert res.cand == int(np.argmax(l[m])) and res.prob == 1.0
            continue
        p_m = sp_softmax(l[m] / cfg.temperature)
        counts = _count_sampled_u(l, cfg, pi, None, V, None)
        assert np.all(np.abs(counts - p_m * LATTICE) <= 1.0 + 1e-6)
        for u in (0.01, 0.4, 0.93):
            res = orc.verify_position(l, cfg, pi, None, 0.5, u)
            assert abs(res.prob - p_m[res.cand]) < 1e-15
        # the draft positions are untouched by the choice of bonus model
        a = orc.verify_position(l, cfg, pi, 2, 0.4, 0.6)
        b = orc.verify_position(l, base, pi, 2, 0.4, 0.6)
        assert (a.accept, a.cand, a.ratio, a.S) == (b.accept, b.cand, b.ratio, b.S)


def test_bonus_probability_is_reported_only_after_gamma_acceptances():
    n, B, V, g = 2, 30, 11, 2
    gen = np.random.default_rng(5)
    logits = gen.normal(size=(n, B, g + 1, V)).astype(np.float32)
    drafts = gen.integers(0, V, size=(B, g))
    for m in (-1, 0, 1):
        cfg = orc.OracleConfig(n=n, combine=WE, weights=[0.5, 0.5], temperature=1.0, gamma=g, vocab=V, bonus_model=m)
        out = orc.verify(logits, "f32", drafts, np.zeros(B, int), cfg, seed=9, offset=3)
        full = out["accept_count"] == g
        assert full.any() and (~full).any()
        assert np.all(np.isnan(out["bonus_prob"][~full]))
        for b in np.nonzero(full)[0]:
            l = logits[:, b, g, :].astype(np.float64)
            law = 0.5 * sp_softmax(l[0]) + 0.5 * sp_softmax(l[1]) if m < 0 else sp_softmax(l[m])
            assert abs(out["bonus_prob"][b] - law[out["out_tokens"][b, g]]) < 1e-14


def test_proposer_per_position_changes_q_position_by_position():
    """Algorithm 2: the cached sequence mixes tokens proposed by different models, so q at position j is
    the law of the model that proposed draft j.  P(accept draft d at j) = min(1, r_j(d) / p_{pi_j, j}(d)),
    counted over the uniform lattice with the laws rebuilt from scipy's softmax."""
    n, V, g = 3, 6, 3
    gen = np.random.default_rng(12)
    logits = (gen.normal(size=(n, 1, g + 1, V)) * 1.5).astype(np.float32)
    w = [0.5, 0.3, 0.2]
    cfg = cfg_we(n, V, w, T=0.9, gamma=g)
    prop = np.array([[2, 0, 1, 0]])
    drafts = np.array([[1, 4, 2]])
    for j in range(g):
        l = logits[:, 0, j, :].astype(np.float64)
        ps = [sp_softmax(l[i] / cfg.temperature) for i in range(n)]
        r = sum(cfg.w64[i] * ps[i] for i in range(n))
        want = min(1.0, r[drafts[0, j]] / ps[prop[0, j]][drafts[0, j]])
        # bisection over the accept decision of the whole-batch entry point at position j
        def accepted(mi):
            ua = np.full((1, g + 1), 2.0 ** -24)     # every other position accepts
            ua[0, j] = lattice_u(mi)
            out = orc.verify(logits, "f32", drafts, prop, cfg, 0, 0, uniforms=(ua, np.full((1, g + 1), 0.5)))
            return bool(out["accept"][0, j])
        lo, hi = 0, LATTICE - 1
        assert accepted(lo)
        if accepted(hi):
            count = LATTICE
        else:
            while hi - lo > 1:
                mid = (lo + hi) // 2
                if accepted(mid):
                    lo = mid
                else:
                    hi = mid
            count = lo + 1
        assert abs(count / LATTICE - want) <= 2.0 ** -22
    # a constant table is the per-row form
    a = orc.verify(logits, "f32", drafts, np.array([[1, 1, 1, 1]]), cfg, 3, 1)
    b = orc.verify(logits, "f32", drafts, np.array([1]), cfg, 3, 1)
    for k in ("accept_count", "out_tokens", "row_status"):
        assert np.array_equal(a[k], b[k])


# --------------------------------------------------------------------------------------
# the disclosed boundary cases, and the conventions for q(x) = 0, an empty residual and
# non-finite logits at T = 0
# --------------------------------------------------------------------------------------
def test_accept_boundary_flag_is_the_1e5_band_around_the_threshold():
    """A position is a disclosed boundary case of the accept test iff |u - min(1, r(x)/q(x))| < 1e-5
    (the band in which an fp32 evaluation of Eq. 6 may decide differently from an fp64 one)."""
    V = 12
    l = rng_logits(41, 2, V)
    cfg = cfg_we(2, V, [0.5, 0.5])
    p0, p1 = sp_softmax(l[0]), sp_softmax(l[1])
    ratios = (0.5 * p0 + 0.5 * p1) / p0
    d = int(np.argmin(np.abs(ratios - 0.8)))          # a draft whose threshold lies strictly inside (0, 1)
    thr = float(ratios[d])
    assert 0.55 < thr < 0.999
    for delta, want in ((0.9e-5, True), (-0.9e-5, True), (1.1e-5, False), (-1.1e-5, False), (0.0, True)):
        res = orc.verify_position(l, cfg, 0, d, thr + delta, 0.5)
        assert res.boundary_accept is want, (delta, res.boundary_accept)
        assert res.accept is (delta <= 0.0)
    # a threshold clipped at 1: the band is measured from 1, not from the ratio
    d1 = int(np.argmax(ratios))
    assert ratios[d1] > 1.0 + 1e-3
    assert orc.verify_position(l, cfg, 0, d1, 1.0 - 0.9e-5, 0.5).boundary_accept
    assert not orc.verify_position(l, cfg, 0, d1, 1.0 - 1.1e-5, 0.5).boundary_accept


def test_sample_boundary_flag_is_the_1e6_band_around_the_normalised_cdf_edges():
    """A drawn token is a disclosed boundary case iff one of its two CDF edges, divided by the total
    mass, lies within 1e-6 of the uniform."""
    V = 9
    l = rng_logits(43, 2, V)
    cfg = cfg_we(2, V, [0.5, 0.5], gamma=0)
    r = 0.5 * sp_softmax(l[0]) + 0.5 * sp_softmax(l[1])
    cdf = np.cumsum(r) / np.sum(r)
    k = 4
    lo, hi = float(cdf[k - 1]), float(cdf[k])
    assert hi - lo > 1e-4                             # the token is wide enough to sit strictly inside
    for u, want_tok, want_flag in ((lo + 0.9e-6, k, True), (lo + 1.1e-6, k, False), (hi - 0.9e-6, k, True),
                                   (hi - 1.1e-6, k, False), (lo - 0.9e-6, k - 1, True), (hi + 0.9e-6, k + 1, True),
                                   (0.5 * (lo + hi), k, False)):
        res = orc.verify_position(l, cfg, 0, None, 0.5, u)
        assert res.cand == want_tok and res.boundary_sample is want_flag, (u, res.cand, res.boundary_sample)
    # the residual's edges are normalised by the residual mass S, not by 1
    cfg1 = cfg_we(2, V, [0.5, 0.5])
    q = sp_softmax(l[0])
    resid = np.maximum(0.0, r - q)
    S = resid.sum()
    assert 0.01 < S < 0.9
    c = np.cumsum(resid) / S
    kk = int(np.argmax(resid))
    lo_r = float(c[kk - 1]) if kk > 0 else 0.0
    assert orc.verify_position(l, cfg1, 0, 0, 0.99999, lo_r + 0.9e-6).boundary_sample
    assert not orc.verify_position(l, cfg1, 0, 0, 0.99999, lo_r + 1.1e-6 + 1e-9).boundary_sample
    assert orc.verify_position(l, cfg1, 0, 0, 0.99999, lo_r + 1.1e-6 + 1e-9).cand == kk


def test_q_zero_convention_ratio_is_infinite_iff_r_is_positive():
    """A convention of this build, not of the paper (which never meets q(x) = 0 because the draft is
    drawn from q): the ratio is +inf when r(x) > 0 (accepted for every u) and 0 otherwise (rejected
    for every u); the position reports Q_ZERO either way.  Reached at T = 0 with a draft that is
    not the proposer's argmax."""
    V = 6
    l = np.zeros((2, V))
    l[0, 1] = 3.0          # proposer's argmax: token 1
    l[1, 4] = 3.0          # the other model's argmax: token 4
    cfg = cfg_we(2, V, [0.5, 0.5], T=0.0)
    for u in (lattice_u(0), lattice_u(LATTICE - 1)):
        res = orc.verify_position(l, cfg, 0, 4, u, 0.5)              # r(4) = 0.5 > 0 = q(4)
        assert res.status == orc.STATUS_Q_ZERO and res.ratio == math.inf and res.accept
        res = orc.verify_position(l, cfg, 0, 2, u, 0.5)              # r(2) = 0 = q(2)
        assert res.status & orc.STATUS_Q_ZERO and res.ratio == 0.0 and not res.accept
        res = orc.verify_position(l, cfg, 0, 1, u, 0.5)              # q(1) = 1: the ordinary branch
        assert res.status == 0 and res.ratio == 0.5
    # whole row: the flag is reported, the accepted draft is kept
    logits = np.broadcast_to(l[:, None, None, :], (2, 1, 2, V)).copy()
    out = orc.verify(logits, "f64", [[4]], [0], cfg, 3, 0)
    assert out["accept_count"][0] == 1 and out["row_status"][0] == orc.STATUS_Q_ZERO


def test_empty_residual_convention_draws_from_r_and_reports_only_on_rejection():
    """A convention of this build: when r and q coincide the residual max(0, r - q) has no mass; in exact
    arithmetic no rejection can then happen, so the case only arises from a bad draft.  The token is
    drawn from r with the same uniform and RESIDUAL_EMPTY is reported only if the position rejected."""
    V = 7
    l = rng_logits(47, 2, V)
    l[1] = l[0]                                                       # both models identical: r == q exactly
    cfg = cfg_we(2, V, [0.5, 0.5])
    p = sp_softmax(l[0])
    cdf = np.cumsum(p)
    for u in (0.1, 0.5, 0.93):
        k_want = int(np.searchsorted(cdf, u * cdf[-1]))
        res = orc.verify_position(l, cfg, 0, V + 3, 0.5, u)           # a bad draft forces the rejection
        assert res.status == (orc.STATUS_BAD_DRAFT | orc.STATUS_RESIDUAL_EMPTY)
        assert res.S == 0.0 and res.cand == k_want
        res = orc.verify_position(l, cfg, 0, 2, 0.5, u)               # accepted (ratio 1): candidate unused, no flag
        assert res.accept and res.status == 0 and res.cand == k_want


def test_greedy_with_non_finite_logits_reports_the_position():
    """T = 0 reading: a NaN or +inf anywhere among the position's logits, or a model (or the masked
    combination) without a finite maximum, makes the one-hot distributions undefined; the position
    then counts as rejected with no candidate.  Logits of -inf are legal as long as a finite maximum remains."""
    V = 8
    base = rng_logits(53, 2, V)
    we, ll = cfg_we(2, V, [0.5, 0.5], T=0.0), cfg_ll(2, V, [1.5, -0.5], T=0.0)
    llm = cfg_ll(2, V, [1.0, -0.5], T=0.0, mask_model=0, alpha=0.1)
    for cfg in (we, ll, llm):
        for bad in (np.nan, np.inf):
            for model in (0, 1):
                l = base.copy()
                l[model, 3] = bad
                r, q, ok = orc.position_distributions(l, cfg, 0)
                assert not ok and np.all(np.isnan(r))
                res = orc.verify_position(l, cfg, 0, 2, 0.5, 0.5)
                assert res.status == orc.STATUS_NONFINITE and not res.accept and res.cand == -1
        l = base.copy()
        k = int(np.argmin(base[0]))                                   # never an argmax, inside no mask
        l[0, k] = -np.inf                                             # ruled-out token: still well defined
        r, q, ok = orc.position_distributions(l, cfg, 0)
        assert ok and q[int(np.argmax(l[0]))] == 1.0 and abs(r.sum() - 1.0) < 1e-15 and r[k] == 0.0
        if cfg is not we:
            l = base.copy()
            l[1, 3] = -np.inf                                         # times a negative weight: a combined logit of +inf
            assert not orc.position_distributions(l, cfg if cfg is ll else ll, 0)[2]
        l = base.copy()
        l[1, :] = -np.inf                                             # a model with no finite maximum
        _, _, ok = orc.position_distributions(l, cfg, 0)
        assert not ok
    # logit level: +inf * negative weight would give -inf - harmless in a max - but the input itself is rejected
    l = base.copy()
    l[1, 5] = np.inf
    assert not orc.position_distributions(l, ll, 0)[2]
    # whole row at T = 0: the non-finite position stops the row and emits -1
    logits = np.broadcast_to(base[:, None, None, :], (2, 1, 3, V)).copy()
    logits[0, 0, 1, 0] = np.nan
    d = int(np.argmax(base[0]))
    out = orc.verify(logits, "f64", [[d, d]], [0], cfg_we(2, V, [0.5, 0.5], T=0.0, gamma=2), 5, 0)
    # position 0: the draft is the proposer's argmax, so r(d) >= 0.5 = ratio and some uniforms accept
    a = int(out["accept_count"][0])
    assert a <= 1
    if a == 1:
        assert out["out_tokens"][0, 1] == -1 and out["row_status"][0] & orc.STATUS_NONFINITE
    else:
        assert out["row_status"][0] == 0
