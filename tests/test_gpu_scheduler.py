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
