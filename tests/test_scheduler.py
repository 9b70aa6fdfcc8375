"""The alternate proposal framework (Sec. 3.3, Algorithm 1) driven by the oracle's verification.

Host logic only: the scheduler gets its verification call from outside, here the float64 oracle.  With
models that ignore their context every position has the same laws, so the paper's closed forms apply:
the output tokens follow the combined distribution (Sec. 3.1, App. A.1), a cycle yields
(1 - alpha^gamma) / (1 - alpha) tokens on average (App. A.2), and all drafts pass with probability
alpha^gamma, in which case the verifier's bonus token opens the next proposal (Thm. 3.4's argument)."""
import numpy as np
import pytest
from scipy.special import softmax as sp_softmax
from scipy.stats import chi2 as chi2_dist

from oracle import cos_oracle as orc
from paper_2502_01662_b200 import scheduler as sch

WE, LL = orc.COMBINE_PROB_ENSEMBLE, orc.COMBINE_LOGIT_LINEAR


def oracle_verify(combine, weights, T, V, mask_model=-1, mask_alpha=1.0):
    def verify(logits, drafts, proposer, bonus_model, seed, offset):
        g = logits.shape[2] - 1
        cfg = orc.OracleConfig(n=2, combine=combine, weights=list(weights), temperature=T, gamma=g, vocab=V,
                               mask_model=mask_model, mask_alpha=mask_alpha, bonus_model=bonus_model)
        out = orc.verify(logits, "f32", drafts, np.array([proposer]), cfg, seed, offset)
        return int(out["accept_count"][0]), out["out_tokens"][0], float(out["bonus_prob"][0])
    return verify


def laws(models, combine, weights, T):
    l = [m.table[0].astype(np.float64) for m in models]
    p = [sp_softmax(x / T) for x in l]
    w = np.asarray(np.asarray(weights, dtype=np.float32), dtype=np.float64)
    r = w[0] * p[0] + w[1] * p[1] if combine == WE else sp_softmax((w[0] * l[0] + w[1] * l[1]) / T)
    return p, r


@pytest.mark.parametrize("combine,weights,gammas", [(WE, (0.5, 0.5), (3, 2)), (WE, (0.3, 0.7), (1, 4)),
                                                    (LL, (1.0, -0.5), (2, 3))])
def test_output_follows_the_combined_law_and_cycles_match_the_closed_forms(combine, weights, gammas):
    V, T, N = 12, 0.9, 16000
    models = sch.make_table_models(2, V, contexts=1, seed=5, sigma=1.2, rho=0.6)
    run = sch.AlternateProposal(models, gammas, T, oracle_verify(combine, weights, T, V), propose_seed=11, verify_seed=12,
                                keep_history=True)
    tokens, st = run.generate([0], N)
    p, r = laws(models, combine, weights, T)
    # every emitted token follows r, although bonus tokens are drawn from one model's own law
    counts = np.bincount(np.asarray(tokens), minlength=V)
    chi2 = float(np.sum((counts - len(tokens) * r) ** 2 / (len(tokens) * r)))
    assert chi2_dist.sf(chi2, V - 1) > 1e-4, (chi2, counts, len(tokens) * r)
    # per proposer: tokens per cycle and the frequency of a full acceptance
    for i in (0, 1):
        alpha = float(np.minimum(p[i], r).sum())            # sum_x q min(1, r/q)
        g = gammas[i]
        cyc = [c for c in st.history if c.proposer == i]
        assert len(cyc) > 300
        n_tok = np.array([len(c.emitted) for c in cyc], dtype=np.float64)
        want = (1 - alpha ** g) / (1 - alpha)
        assert abs(n_tok.mean() - want) < 4.5 * n_tok.std() / np.sqrt(len(cyc)) + 1e-9, (i, n_tok.mean(), want)
        full = np.mean([c.accept_count == g for c in cyc])
        sd = np.sqrt(alpha ** g * (1 - alpha ** g) / len(cyc))
        assert abs(full - alpha ** g) < 4.5 * sd + 1e-9, (i, full, alpha ** g)


def test_roles_swap_after_a_full_acceptance_and_reset_after_a_rejection():
    V, T = 40, 1.0
    models = sch.make_table_models(2, V, contexts=16, seed=9)
    gammas = (3, 2)
    run = sch.AlternateProposal(models, gammas, T, oracle_verify(WE, (0.5, 0.5), T, V), keep_history=True)
    tokens, st = run.generate([3, 1], 600)
    assert tokens == [t for c in st.history for t in c.emitted]
    saw_swap = saw_reset = False
    for prev, cur in zip(st.history, st.history[1:]):
        g_prev = gammas[prev.proposer]
        if prev.accept_count == g_prev:
            # the verifier's bonus token is cached and opens the verifier's own proposal
            assert prev.bonus is not None and cur.proposer == 1 - prev.proposer
            assert cur.cached == 1 and cur.drafts[0] == prev.bonus
            assert prev.emitted == prev.drafts            # the bonus itself is not emitted
            saw_swap = True
        else:
            assert prev.bonus is None and cur.proposer == 0 and cur.cached == 0
            assert len(prev.emitted) == prev.accept_count + 1
            assert prev.emitted[:-1] == prev.drafts[: prev.accept_count]
            saw_reset = True
    assert saw_swap and saw_reset
    # forward passes: the proposer generates gamma - cached tokens, the verifier scores once per cycle
    assert st.proposed == sum(gammas[c.proposer] - c.cached for c in st.history)
    assert st.scored == st.cycles == len(st.history)
    assert models[0].calls + models[1].calls == st.proposed + st.scored


def test_greedy_run_is_the_argmax_chain_of_the_combined_model():
    """T = 0: every distribution is one-hot, so the output is the greedy decoding of the combined model
    (here the ensemble's heaviest atom: with weights 0.3 / 0.7 that is model 1's argmax)."""
    V = 30
    models = sch.make_table_models(2, V, contexts=8, seed=21)
    run = sch.AlternateProposal(models, (2, 3), 0.0, oracle_verify(WE, (0.3, 0.7), 0.0, V))
    tokens, _ = run.generate([5], 60)
    S = [5]
    for t in tokens:
        a0, a1 = int(np.argmax(models[0].logits(S))), int(np.argmax(models[1].logits(S)))
        # r = 0.3 onehot(a0) + 0.7 onehot(a1): a rejected draft is replaced by the residual's first atom in
        # token order, an accepted one is either atom; both are atoms of r
        assert t in (a0, a1)
        S.append(t)


# --------------------------------------------------------------------------------------
# n models (Algorithm 2)
# --------------------------------------------------------------------------------------
def oracle_verify_n(n, combine, weights, T, V):
    def verify(logits, drafts, proposer, bonus_model, seed, offset):
        g = logits.shape[2] - 1
        cfg = orc.OracleConfig(n=n, combine=combine, weights=list(weights), temperature=T, gamma=g, vocab=V,
                               bonus_model=bonus_model)
        prop = np.array([proposer]) if np.isscalar(proposer) else np.asarray(proposer)
        out = orc.verify(logits, "f32", drafts, prop, cfg, seed, offset)
        return int(out["accept_count"][0]), out["out_tokens"][0], float(out["bonus_prob"][0])
    return verify


def test_three_models_follow_the_walk_through_of_the_paper():
    """App. B, proposal lengths (3, 2, 1): M1 proposes x1..x3; M2 scores them, draws x4 and proposes x5; M3
    scores x1..x5 and draws x6; now x1..x3 have been scored by all three and are verified together.  If they
    pass, M1 (which holds no probabilities for x4..x6) scores those three and proposes x7..x9, after which x4
    and x5 are verifiable."""
    V, T = 50, 1.0
    models = sch.make_table_models(3, V, contexts=32, seed=4, sigma=0.3, rho=0.95)   # near-identical: drafts pass
    run = sch.CollaborativeSpeculation(models, (3, 2, 1), T, oracle_verify_n(3, WE, (0.4, 0.3, 0.3), T, V), keep_events=True)
    run.generate([7], 12)
    ev = [(e.kind, e.model, e.count) for e in run.events]
    assert ev[:5] == [("propose", 0, 3), ("score", 1, 3), ("propose", 1, 1), ("score", 2, 5), ("verify", -1, 3)]
    first = run.events[4]
    if first.accepted == 3:
        assert ev[5:10] == [("propose", 2, 0), ("score", 0, 3), ("verify", -1, 2), ("propose", 0, 2), ("score", 1, 4)] or \
            ev[5:8] == [("propose", 2, 0), ("score", 0, 3), ("verify", -1, 2)]
    else:
        assert ev[5] == ("propose", 0, 3)       # everything cached was dropped: the default proposer again


@pytest.mark.parametrize("n,weights,gammas", [(3, (0.5, 0.3, 0.2), (3, 2, 1)), (2, (0.5, 0.5), (2, 2)),
                                              (4, (0.25, 0.25, 0.25, 0.25), (1, 2, 1, 3))])
def test_n_model_output_follows_the_combined_law(n, weights, gammas):
    """Every emitted token passed the accept test against r = sum_i w_i p_i with the law of its own proposer
    as q (or was resampled from the residual), whichever model produced it and whether it began as a bonus
    token: with context-free models the output is an i.i.d. sample of r."""
    V, T, N = 10, 1.1, 12000
    models = sch.make_table_models(n, V, contexts=1, seed=17, sigma=1.0, rho=0.5)
    run = sch.CollaborativeSpeculation(models, gammas, T, oracle_verify_n(n, WE, weights, T, V), propose_seed=5,
                                       verify_seed=6, keep_events=True)
    tokens, st = run.generate([0], N)
    w = np.asarray(np.asarray(weights, dtype=np.float32), dtype=np.float64)
    r = sum(w[i] * sp_softmax(models[i].table[0].astype(np.float64) / T) for i in range(n))
    counts = np.bincount(np.asarray(tokens[:N]), minlength=V)
    chi2 = float(np.sum((counts - N * r) ** 2 / (N * r)))
    assert chi2_dist.sf(chi2, V - 1) > 1e-4, (chi2, counts, N * r)
    # every model proposed and scored; forward passes are all accounted for
    kinds = {(e.kind, e.model) for e in run.events}
    assert all(("score", i) in kinds for i in range(1, n)) and ("propose", 0) in kinds
    assert sum(m.calls for m in models) == st.proposed + st.scored
    # a verification never covers more tokens than the cache held, and after a rejection the default proposer restarts
    for prev, cur in zip(run.events, run.events[1:]):
        if prev.kind == "verify" and prev.accepted < prev.count:
            assert (cur.kind, cur.model, cur.count) == ("propose", 0, gammas[0])
