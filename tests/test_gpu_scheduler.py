"""The alternate proposal framework (Algorithm 1) with the CUDA library as its verification call: the token
stream must be the one the float64 oracle produces in the same place, cycle by cycle."""
import numpy as np
import pytest

from oracle import cos_oracle as orc
from paper_2502_01662_b200 import scheduler as sch

from test_scheduler import oracle_verify

pytestmark = pytest.mark.gpu

WE, LL = orc.COMBINE_PROB_ENSEMBLE, orc.COMBINE_LOGIT_LINEAR


@pytest.mark.parametrize("combine,weights,T,gammas", [(WE, (0.5, 0.5), 0.8, (4, 2)), (LL, (1.5, -0.5), 1.0, (3, 3)),
                                                      (WE, (0.4, 0.6), 0.0, (2, 3))])
def test_gpu_driven_stream_equals_oracle_driven_stream(combine, weights, T, gammas):
    V, N = 4099, 400                      # a ragged vocabulary; a few hundred cycles
    def run_with(verify):
        models = sch.make_table_models(2, V, contexts=64, seed=33, sigma=2.5, rho=0.85)
        run = sch.AlternateProposal(models, gammas, T, verify, propose_seed=3, verify_seed=4, keep_history=True)
        return run.generate([1, 2, 3], N)
    gpu_fn = sch.gpu_verify(combine, weights, T, V)
    try:
        got, st_g = run_with(gpu_fn)
    finally:
        gpu_fn.close()
    want, st_o = run_with(oracle_verify(combine, weights, T, V))
    assert got == want
    assert [c.accept_count for c in st_g.history] == [c.accept_count for c in st_o.history]
    assert [c.bonus for c in st_g.history] == [c.bonus for c in st_o.history]
    # both kinds of cycle occurred
    assert any(c.bonus is not None for c in st_g.history) and any(c.bonus is None for c in st_g.history)


from test_scheduler import oracle_verify_n


@pytest.mark.parametrize("n,combine,weights,T,gammas", [(3, WE, (0.5, 0.3, 0.2), 0.9, (3, 2, 1)),
                                                        (2, LL, (1.0, -0.5), 1.0, (2, 3)),
                                                        (4, WE, (0.1, 0.2, 0.3, 0.4), 0.0, (2, 1, 2, 1))])
def test_n_model_stream_on_the_gpu_equals_the_oracle_driven_stream(n, combine, weights, T, gammas):
    """Algorithm 2 with the CUDA library behind `verify`: proposer tables, bonus tokens drawn from a named
    model (gamma = 0 calls) and verified prefixes of varying length, against the oracle in the same place."""
    V, N = 3000, 300
    def run_with(verify):
        models = sch.make_table_models(n, V, contexts=64, seed=41, sigma=2.0, rho=0.9)
        run = sch.CollaborativeSpeculation(models, gammas, T, verify, propose_seed=8, verify_seed=9, keep_events=True)
        toks, _ = run.generate([4, 4], N)
        return toks, [(e.kind, e.model, e.count, e.accepted) for e in run.events]
    gpu_fn = sch.gpu_verify(combine, weights, T, V)
    try:
        got, ev_g = run_with(gpu_fn)
    finally:
        gpu_fn.close()
    want, ev_o = run_with(oracle_verify_n(n, combine, weights, T, V))
    assert got == want and ev_g == ev_o
    assert any(k == "verify" and a == c for k, _, c, a in ev_g) and any(k == "verify" and a < c for k, _, c, a in ev_g)
