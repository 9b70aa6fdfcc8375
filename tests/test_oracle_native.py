"""The C++ oracle must give the rows of the Python oracle (which carries the pins against the paper): integer
outputs identical, floating-point diagnostics to 1e-12.  Both are test infrastructure; they share no code."""
import numpy as np
import pytest

from oracle import cos_oracle as orc
from oracle import cos_oracle_native as nat
from paper_2502_01662_b200 import synth

CASES = {
    "cfg1": dict(batch=3, vocab=1000, gamma=3),
    "cfg2": dict(batch=6, vocab=777, gamma=4),
    "cfg3": dict(batch=5, vocab=1544, gamma=5),
    "cfg3_f16": dict(batch=4, vocab=1003, gamma=2),
    "cfg4": dict(batch=8, vocab=999, gamma=3),
    "cfg5": dict(batch=4, vocab=2048, gamma=4),
    "cfg5_greedy": dict(batch=6, vocab=2001, gamma=4),
}


def oracle_cfg(w, bonus_model=-1):
    return orc.OracleConfig(n=w.n, combine=w.combine, weights=list(w.weights), temperature=w.temperature, gamma=w.gamma,
                            vocab=w.vocab, mask_model=w.mask_model, mask_alpha=w.mask_alpha, bonus_model=bonus_model)


def same(a, b, rows=None):
    for k in ("accept_count", "out_tokens", "row_status", "accept", "cand", "boundary_accept", "boundary_sample", "pos_status"):
        x, y = np.asarray(a[k]), np.asarray(b[k])
        if rows is not None:
            x, y = x[list(rows)], y[list(rows)]
        assert np.array_equal(x, y), k
    for k in ("ratio", "r_d", "q_d", "S", "bonus_prob", "u_acc", "u_smp"):
        x, y = np.asarray(a[k], dtype=np.float64), np.asarray(b[k], dtype=np.float64)
        if rows is not None:
            x, y = x[list(rows)], y[list(rows)]
        assert np.array_equal(np.isnan(x), np.isnan(y)), k
        np.testing.assert_allclose(x, y, rtol=1e-12, atol=1e-13, equal_nan=True, err_msg=k)   # S is a sum of differences


@pytest.mark.parametrize("name", sorted(CASES))
def test_native_oracle_gives_the_python_oracles_rows(name):
    w = synth.CONFIGS[name].scaled(**CASES[name])
    inp = synth.make_inputs(w, "cpu")
    host = synth.logits_as_numpy(inp["logits"])
    d, p = inp["drafts"].numpy(), inp["proposer"].numpy()
    ref = orc.verify(host, w.dtype, d, p, oracle_cfg(w), inp["seed"], 7, row_base=11)
    got = nat.verify(host, w.dtype, d, p, oracle_cfg(w), inp["seed"], 7, row_base=11)
    same(ref, got)
    # a subset of rows, on one thread and on several
    rows = [w.batch - 1, 0]
    for threads in (1, 3):
        part = nat.verify(host, w.dtype, d, p, oracle_cfg(w), inp["seed"], 7, row_base=11, rows=rows, threads=threads)
        same(ref, part, rows)


def test_native_oracle_alternate_proposals_bad_drafts_and_non_finite_logits():
    w = synth.CONFIGS["cfg4"].scaled(batch=6, vocab=500, gamma=3)
    inp = synth.make_inputs(w, "cpu")
    host = synth.logits_as_numpy(inp["logits"]).copy()
    d = inp["drafts"].numpy().copy()
    d[1, 0] = w.vocab + 5                      # bad draft
    d[2, 1] = -1
    host[0, 3, 1, 17] = 0x7FC0                 # NaN (bf16 pattern) at row 3, position 1
    host[1, 4, 0, 5] = 0xFF80                  # -inf: legal in the ensemble
    g = np.random.default_rng(5)
    table = g.integers(0, w.n, size=(w.batch, w.gamma + 1)).astype(np.int32)
    for bonus in (-1, 2):
        ref = orc.verify(host, w.dtype, d, table, oracle_cfg(w, bonus), 99, 3)
        got = nat.verify(host, w.dtype, d, table, oracle_cfg(w, bonus), 99, 3)
        same(ref, got)
    assert ref["row_status"][1] & orc.STATUS_BAD_DRAFT


def test_native_oracle_greedy_ties_and_identical_models():
    V = 64
    l = np.zeros((2, 2, 2, V), np.float32)
    l[0, :, :, [5, 9]] = 2.0                   # ties: the lowest index wins
    l[1, :, :, [9, 30]] = 2.0
    for combine, wts in ((orc.COMBINE_PROB_ENSEMBLE, [0.5, 0.5]), (orc.COMBINE_LOGIT_LINEAR, [1.0, 1.0])):
        cfg = orc.OracleConfig(n=2, combine=combine, weights=wts, temperature=0.0, gamma=1, vocab=V)
        ref = orc.verify(l, "f32", [[5], [9]], [0, 1], cfg, 1, 0)
        got = nat.verify(l, "f32", [[5], [9]], [0, 1], cfg, 1, 0)
        same(ref, got)
    # identical models at T > 0: r == q, nothing rejects, the residual is empty
    l[1] = l[0]
    cfg = orc.OracleConfig(n=2, combine=orc.COMBINE_PROB_ENSEMBLE, weights=[0.5, 0.5], temperature=1.0, gamma=1, vocab=V)
    ref = orc.verify(l, "f32", [[5], [V + 1]], [0, 1], cfg, 1, 0)
    got = nat.verify(l, "f32", [[5], [V + 1]], [0, 1], cfg, 1, 0)
    same(ref, got)
    assert got["row_status"][1] == (orc.STATUS_BAD_DRAFT | orc.STATUS_RESIDUAL_EMPTY)
