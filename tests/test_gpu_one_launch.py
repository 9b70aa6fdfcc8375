"""The one-launch form of a run (cos_verify_set_one_launch) against the oracle, and its bounded waits."""
import numpy as np
import pytest
import torch

import helpers
from paper_2502_01662_b200 import COS_ROW_BAD_DRAFT, COS_ROW_NONFINITE, COS_ROW_RESIDUAL_EMPTY, CosVerifyError, synth
from paper_2502_01662_b200.binding import COS_ROW_FAULT

pytestmark = pytest.mark.gpu
C = synth.CONFIGS


def one_launch_verifier(w, form=1, **kw):
    """form 1: the whole run in one launch; form 2: staged streaming launch, tokens drawn by the persistent kernel."""
    v = helpers.make_verifier(w, **kw)
    v.set_one_launch(form)
    info = v.info()
    assert (info["one_launch"] and info["launches_per_run"] == 1) if form == 1 else (info["draw_items"] and info["launches_per_run"] == 2)
    return v


def we(n, weights, dtype="bf16", T=1.0, **kw):
    return synth.Workload(f"we{n}_{dtype}", n, 0, weights, T, kw.get("batch", 6), kw.get("gamma", 4), kw.get("vocab", 20008),
                          dtype, "gauss", sigma=2.5, rho=0.7, proposer_rule="cycle")


SMALL = [
    C["cfg3"].scaled(batch=7, vocab=20008, gamma=5, name="we2_zipf"),
    C["cfg3_f16"].scaled(batch=5, vocab=9000, gamma=3, name="we2_f16"),
    C["cfg1"].scaled(batch=3, vocab=32000, gamma=4, name="we2_f32"),
    we(1, (1.0,)), we(3, (0.5, 0.3, 0.2)), we(4, (0.4, 0.3, 0.2, 0.1), dtype="f32", vocab=12004),
    C["cfg4"].scaled(batch=6, vocab=128256, gamma=2, name="we4_chunks"),        # several streaming chunks per position
    C["cfg5"].scaled(batch=5, vocab=50000, gamma=3, name="ll2"),
    C["cfg5"].scaled(batch=3, vocab=256000, gamma=2, name="ll2_chunks"),
    synth.Workload("ll3", 3, 1, (1.2, -0.4, 0.2), 0.9, 5, 3, 16000, "bf16", "gauss", sigma=2.0, rho=0.6, proposer_rule="cycle"),
    C["cfg3"].scaled(batch=4, vocab=151936, gamma=0, name="gamma0"),            # direct sampling from r
    C["cfg3"].scaled(batch=3, vocab=4096, gamma=15, name="gamma15"),            # sixteen positions: the row word is full
]


@pytest.mark.parametrize("form", [1, 2])
@pytest.mark.parametrize("w", SMALL, ids=[w.name for w in SMALL])
def test_one_launch_matches_the_oracle(w, form):
    inputs = synth.make_inputs(w, "cuda")
    v = one_launch_verifier(w, form)
    try:
        gpu = helpers.run_gpu(w, inputs, verifier=v, diag=True)
        again = helpers.run_gpu(w, inputs, verifier=v, diag=True)      # the scratch was left clean; results do not depend on scheduling
    finally:
        v.close()
    ref = helpers.run_oracle(w, inputs, native=True)
    stats = helpers.check_parity(w, gpu, ref)
    assert stats["excused_accept"] + stats["excused_sample"] <= 1, stats
    for k in ("accept_count", "out_tokens", "row_status"):
        assert np.array_equal(gpu[k], again[k]), k
    assert np.array_equal(gpu["diag"], again["diag"], equal_nan=True)
    a = gpu["accept_count"]
    assert np.all(gpu["out_tokens"][np.arange(w.batch), a] >= 0)
    # the residual mass is reported where a token was drawn from the residual
    for b in range(w.batch):
        if a[b] < w.gamma:
            np.testing.assert_allclose(gpu["diag"][b, a[b], 3], ref["S"][b, a[b]], rtol=1e-5, atol=1e-7)


@pytest.mark.parametrize("form", [1, 2])
@pytest.mark.parametrize("name,nrows", [("cfg3", 64), ("cfg4", 32), ("cfg5", 32)])
def test_one_launch_full_size(name, nrows, form):
    w = C[name]
    inputs = synth.make_inputs(w, "cuda")
    rows = sorted(np.random.default_rng(5).choice(w.batch, size=min(nrows, w.batch), replace=False).tolist())
    v = one_launch_verifier(w, form)
    try:
        gpu = helpers.run_gpu(w, inputs, verifier=v, diag=True)
        again = helpers.run_gpu(w, inputs, verifier=v)
        v.set_one_launch(False)                                          # the staged form on the same context
        staged = helpers.run_gpu(w, inputs, verifier=v)
    finally:
        v.close()
    ref = helpers.run_oracle(w, inputs, rows=rows, native=True)
    stats = helpers.check_parity(w, gpu, ref, rows=rows)
    assert stats["excused_accept"] + stats["excused_sample"] <= 2, stats
    for k in ("accept_count", "out_tokens", "row_status"):
        assert np.array_equal(gpu[k], again[k]), k
    # the two forms may only differ in rows the oracle marks as boundary cases
    diff = [b for b in range(w.batch) if not np.array_equal(gpu["out_tokens"][b], staged["out_tokens"][b])]
    assert len(diff) <= 2, diff
    del inputs
    torch.cuda.empty_cache()


def test_one_launch_alternate_proposals_and_bonus_model():
    w = C["cfg4"].scaled(batch=8, vocab=12808, gamma=3, name="alt")
    inputs = synth.make_inputs(w, "cuda")
    g = np.random.default_rng(3)
    table = torch.as_tensor(g.integers(0, w.n, size=(w.batch, w.gamma + 1)).astype(np.int32), device="cuda")
    drafts = inputs["drafts"].clone()
    # drafts that every model likes, so that some rows reach the bonus position
    drafts[:4] = torch.argmax(inputs["logits"][0, :4, : w.gamma].float(), dim=-1).to(torch.int32)
    mod = dict(inputs, proposer=table, drafts=drafts)
    for bonus in (-1, 2):
        ref = helpers.run_oracle(w, mod, bonus_model=bonus, native=True)
        for form in (1, 2):
            v = one_launch_verifier(w, form)
            try:
                gpu = helpers.run_gpu(w, mod, verifier=v, diag=True, bonus_model=bonus if bonus >= 0 else None)
            finally:
                v.close()
            helpers.check_parity(w, gpu, ref)


def test_one_launch_bad_drafts_non_finite_logits_and_empty_residual():
    w = C["cfg3"].scaled(batch=6, vocab=8192, gamma=3, name="edges")
    inputs = synth.make_inputs(w, "cuda")
    logits, drafts = inputs["logits"].clone(), inputs["drafts"].clone()
    drafts[0, 0] = w.vocab + 3
    drafts[1, 1] = -2
    logits[0, 2, 0, 77] = float("nan")
    logits[1, 3, 1, 5] = float("inf")
    logits[0, 4, :, 9] = float("-inf")           # legal in the ensemble
    logits[1, 5] = logits[0, 5]                  # identical models: r == q, the residual is empty
    drafts[5, 0] = w.vocab                       # ... and a bad draft forces a token all the same
    mod = dict(inputs, logits=logits, drafts=drafts)
    ref = helpers.run_oracle(w, mod, native=True)
    for form in (2, 1):
        v = one_launch_verifier(w, form)
        try:
            gpu = helpers.run_gpu(w, mod, verifier=v, diag=True)
        finally:
            v.close()
        helpers.check_parity(w, gpu, ref)
    assert gpu["row_status"][0] & COS_ROW_BAD_DRAFT
    assert gpu["row_status"][2] & COS_ROW_NONFINITE and gpu["out_tokens"][2, 0] == -1
    assert gpu["row_status"][5] == (COS_ROW_BAD_DRAFT | COS_ROW_RESIDUAL_EMPTY)
    assert 0 <= gpu["out_tokens"][5, 0] < w.vocab


@pytest.mark.parametrize("form", [1, 2])
def test_one_launch_partial_batches_strides_and_row_base(form):
    """A context sized for more rows than a run passes, logits that are a strided view, and a row offset."""
    w = C["cfg3"].scaled(batch=5, vocab=20008, gamma=3, name="layout_one_launch")
    inputs = synth.make_inputs(w, "cuda")
    n, B, P, V = inputs["logits"].shape
    padded = torch.zeros((n, B, P + 1, V + 64), dtype=inputs["logits"].dtype, device="cuda")
    padded[:, :, :P, :V] = inputs["logits"]
    view = padded[:, :, :P, :V]                       # same values, other strides (rows still 16-byte aligned)
    v = one_launch_verifier(w, form, max_batch=16)
    try:
        outs = v.run(view, inputs["drafts"], inputs["proposer"], inputs["seed"], inputs["offset"], row_base=1000, diag=True)
        torch.cuda.synchronize()
        gpu = {k: t.cpu().numpy() for k, t in outs.items()}
    finally:
        v.close()
    ref = helpers.run_oracle(w, inputs, row_base=1000, native=True)
    helpers.check_parity(w, gpu, ref)


def test_one_launch_is_refused_where_it_does_not_apply():
    for w in (C["cfg2"].scaled(batch=2, vocab=4096, gamma=2), C["cfg5_greedy"].scaled(batch=2, vocab=4096, gamma=2),
              C["cfg3"].scaled(batch=2, vocab=4100, gamma=2)):
        v = helpers.make_verifier(w)
        try:
            with pytest.raises(CosVerifyError):
                v.set_one_launch(True)
            assert not v.info()["one_launch"]
        finally:
            v.close()


def test_a_wait_that_runs_out_reports_a_fault_and_leaves_the_device_usable():
    """Every wait of the one-launch kernel is a bounded poll.  The test hook keeps one warp's report back, so the
    waits of one block run out: the run must end by itself with COS_ROW_FAULT on every row, and later runs (on the
    same context once the hook is off, and on a fresh one) must be correct.  Nothing traps, hangs or faults."""
    w = C["cfg3"].scaled(batch=8, vocab=20008, gamma=3, name="fault")
    inputs = synth.make_inputs(w, "cuda")
    ref = helpers.run_oracle(w, inputs, native=True)
    v = one_launch_verifier(w)
    try:
        v.set_wait_limit(4096, test_drop_report=True)            # about a millisecond of patience
        bad = helpers.run_gpu(w, inputs, verifier=v)
        assert np.all(bad["row_status"] & COS_ROW_FAULT), bad["row_status"]
        v.set_wait_limit(1 << 20, test_drop_report=False)
        good = helpers.run_gpu(w, inputs, verifier=v, diag=True)
        helpers.check_parity(w, good, ref)
        assert not np.any(good["row_status"] & COS_ROW_FAULT)
    finally:
        v.close()
    fresh = one_launch_verifier(w)
    try:
        helpers.check_parity(w, helpers.run_gpu(w, inputs, verifier=fresh, diag=True), ref)
    finally:
        fresh.close()
