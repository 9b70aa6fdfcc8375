"""GPU parity at the full benchmark sizes (sampled rows) and on the edge cases of the method."""
import numpy as np
import pytest
import torch

import helpers
from paper_2502_01662_b200 import (COS_ROW_BAD_DRAFT, COS_ROW_NONFINITE, COS_ROW_Q_ZERO, COS_ROW_RESIDUAL_EMPTY,
                                   COS_RUN_ALL_RESIDUALS, COS_RUN_INPUTS_SETTLED, CosVerifier, CosVerifyError, synth)
from oracle import cos_oracle as orc

pytestmark = pytest.mark.gpu
C = synth.CONFIGS


@pytest.mark.parametrize("name,nrows", [("cfg1", 1), ("cfg2", 8), ("cfg3", 64), ("cfg4", 32), ("cfg5", 48), ("cfg5_greedy", 48)])
def test_full_size_workloads(name, nrows):
    """The launch configuration bench.py times (default cluster choice, full batch), compared with the
    oracle's C++ twin on every row (workloads 1 to 4) or on a seeded sample of rows (the 2.4 GB workload 5);
    a row's result does not depend on the other rows."""
    w = C[name]
    inputs = synth.make_inputs(w, "cuda")
    rows = sorted(np.random.default_rng(7).choice(w.batch, size=min(nrows, w.batch), replace=False).tolist())
    gpu = helpers.run_gpu(w, inputs, diag=True)
    ref = helpers.run_oracle(w, inputs, rows=rows, native=True)
    stats = helpers.check_parity(w, gpu, ref, rows=rows)
    assert stats["excused_accept"] + stats["excused_sample"] <= 2, stats
    # the rows are not degenerate: some rows reject, and sampling modes do not reject everything at 0
    acc = gpu["accept_count"]
    assert acc.min() >= 0 and acc.max() <= w.gamma
    assert np.all(gpu["out_tokens"][np.arange(w.batch), acc] >= 0)
    # second run with the same arguments is bit-identical (no dependence on scheduling)
    again = helpers.run_gpu(w, inputs, diag=True)
    for k in ("accept_count", "out_tokens", "row_status"):
        assert np.array_equal(gpu[k], again[k]), k
    # four calls queued without a pause on inputs that were complete long before (COS_RUN_INPUTS_SETTLED: a call's
    # streaming launch overlaps the end of the previous call's drawing launch): every one gives the same rows
    v = helpers.make_verifier(w)
    try:
        queued = [v.run(inputs["logits"], inputs["drafts"], inputs["proposer"], inputs["seed"], inputs["offset"],
                        flags=COS_RUN_INPUTS_SETTLED) for _ in range(4)]
        torch.cuda.synchronize()
        for outs in queued:
            for k in ("accept_count", "out_tokens", "row_status"):
                assert np.array_equal(gpu[k], outs[k].cpu().numpy()), k
    finally:
        v.close()
    del inputs
    torch.cuda.empty_cache()


def _small(cfg, **kw):
    return C[cfg].scaled(**kw)


@pytest.mark.parametrize("name,kw", [("cfg3", dict(batch=100, gamma=1)), ("cfg5", dict(batch=80, gamma=1)),
                                     ("cfg3", dict(batch=300, vocab=40000, gamma=1))])
def test_batches_that_do_not_fill_whole_waves(name, kw):
    """Between one and two drawing positions per multiprocessor (and more than two): the one-sweep drawing
    stage then splits a position over more blocks than the device holds at once; every row against the oracle
    on a sample, the residual mass it reports against the oracle's."""
    w = C[name].scaled(name=f"{name}_b{kw['batch']}", **kw)
    inputs = synth.make_inputs(w, "cuda")
    rows = sorted(np.random.default_rng(11).choice(w.batch, size=24, replace=False).tolist())
    gpu = helpers.run_gpu(w, inputs, diag=True)
    ref = helpers.run_oracle(w, inputs, rows=rows)
    stats = helpers.check_parity(w, gpu, ref, rows=rows)
    assert stats["excused_accept"] + stats["excused_sample"] <= 1, stats
    acc = gpu["accept_count"]
    assert np.all(gpu["out_tokens"][np.arange(w.batch), acc] >= 0)
    again = helpers.run_gpu(w, inputs, diag=True)
    for k in ("accept_count", "out_tokens", "row_status"):
        assert np.array_equal(gpu[k], again[k]), k
    del inputs
    torch.cuda.empty_cache()


def test_statistics_of_acceptance_match_eq7():
    """Mean accept flag against mean alpha_j = 1 - sum max(0, r - q) (Eq. 7) from the kernel's own S."""
    w = _small("cfg4", batch=32, vocab=12808, gamma=6, name="stat")
    inputs = synth.make_inputs(w, "cuda")
    gpu = helpers.run_gpu(w, inputs, diag=True, flags=COS_RUN_ALL_RESIDUALS)
    ref = helpers.run_oracle(w, inputs)
    S = gpu["diag"][:, : w.gamma, 3]
    assert np.all(np.isfinite(S))
    np.testing.assert_allclose(S, ref["S"][:, : w.gamma], rtol=1e-5, atol=1e-7)
    alpha = 1.0 - S
    assert np.all(alpha >= np.asarray(w.weights)[inputs["proposer"].cpu().numpy()][:, None] - 1e-6)   # Thm 3.2


def test_row_base_and_partial_batches_and_strides():
    w = _small("cfg3", batch=6, vocab=4096, gamma=3, name="layout")
    inputs = synth.make_inputs(w, "cuda")
    full = helpers.run_gpu(w, inputs)
    # rows 2..5 as a shard: same numbers when row_base = 2; context sized for a larger batch
    v = helpers.make_verifier(w, max_batch=16)
    try:
        part = v.run(inputs["logits"][:, 2:], inputs["drafts"][2:].contiguous(), inputs["proposer"][2:].contiguous(),
                     inputs["seed"], inputs["offset"], row_base=2)
        torch.cuda.synchronize()
        for k in ("accept_count", "out_tokens", "row_status"):
            assert np.array_equal(part[k].cpu().numpy(), full[k][2:]), k
        # a padded layout (row pitch larger than V, still 16-byte aligned) and an unaligned one (scalar loads)
        for pad in (8, 3):
            big = torch.zeros((w.n, w.batch, w.gamma + 1, w.vocab + pad), dtype=inputs["logits"].dtype, device="cuda")
            big[..., : w.vocab] = inputs["logits"]
            view = big[..., : w.vocab]
            got = v.run(view, inputs["drafts"], inputs["proposer"], inputs["seed"], inputs["offset"])
            torch.cuda.synchronize()
            for k in ("accept_count", "out_tokens", "row_status"):
                assert np.array_equal(got[k].cpu().numpy(), full[k]), (pad, k)
    finally:
        v.close()


def test_host_pointer_entry_matches_device_entry():
    w = _small("cfg2", batch=5, vocab=8000, gamma=3, name="host")
    dev_in = synth.make_inputs(w, "cuda")
    want = helpers.run_gpu(w, dev_in, diag=True)
    v = helpers.make_verifier(w, host_staging=True)
    try:
        got = v.run_host(dev_in["logits"].cpu().contiguous().pin_memory(), dev_in["drafts"].cpu().pin_memory(),
                         dev_in["proposer"].cpu().pin_memory(), dev_in["seed"], dev_in["offset"], diag=True)
        for k in ("accept_count", "out_tokens", "row_status"):
            assert np.array_equal(got[k].numpy(), want[k]), k
        np.testing.assert_array_equal(got["diag"].numpy()[..., :3], want["diag"][..., :3])
    finally:
        v.close()


def test_data_dependent_problems_are_flagged_not_trapped():
    w = _small("cfg3", batch=6, vocab=2048, gamma=3, name="flags")
    inputs = synth.make_inputs(w, "cuda")
    logits = inputs["logits"].clone()
    drafts = inputs["drafts"].clone()
    logits[1, 0, 0, 77] = float("nan")          # row 0: NaN at position 0
    logits[0, 1, 1, 5] = float("inf")           # row 1: +inf at position 1
    logits[1, 2, 0, 9] = float("-inf")          # row 2: a token one model rules out (legal)
    drafts[3, 0] = w.vocab                      # row 3: draft outside the vocabulary
    drafts[4, 1] = -1                           # row 4: negative draft at position 1
    bad = dict(inputs, logits=logits, drafts=drafts)
    gpu = helpers.run_gpu(w, bad, diag=True)
    ref = helpers.run_oracle(w, bad)
    helpers.check_parity(w, gpu, ref, check_diag=False)
    assert gpu["row_status"][0] & COS_ROW_NONFINITE and gpu["accept_count"][0] == 0 and gpu["out_tokens"][0, 0] == -1
    assert gpu["row_status"][3] & COS_ROW_BAD_DRAFT and gpu["accept_count"][3] == 0
    assert gpu["row_status"][2] == ref["row_status"][2]


def test_identical_models_accept_everything_and_empty_residual_falls_back_to_r():
    w = _small("cfg3", batch=4, vocab=3000, gamma=2, name="same")
    inputs = synth.make_inputs(w, "cuda")
    logits = inputs["logits"].clone()
    logits[1] = logits[0]                        # r == q exactly
    drafts = inputs["drafts"].clone()
    drafts[2, 0] = w.vocab + 5                   # an invalid draft is rejected although the residual is empty
    same = dict(inputs, logits=logits, drafts=drafts)
    gpu = helpers.run_gpu(w, same, diag=True)
    ref = helpers.run_oracle(w, same)
    helpers.check_parity(w, gpu, ref, check_diag=False)
    assert np.all(gpu["accept_count"][[0, 1, 3]] == w.gamma)
    assert gpu["accept_count"][2] == 0
    assert gpu["row_status"][2] == (COS_ROW_BAD_DRAFT | COS_ROW_RESIDUAL_EMPTY)
    assert 0 <= gpu["out_tokens"][2, 0] < w.vocab


def test_greedy_ensemble_atoms_and_q_zero():
    w = synth.Workload("we_greedy", 3, 0, (0.5, 0.3, 0.2), 0.0, 8, 3, 5000, "f32", "gauss", sigma=2.0, rho=0.5,
                       proposer_rule="cycle")
    inputs = synth.make_inputs(w, "cuda")
    drafts = inputs["drafts"].clone()
    drafts[0, 0] = (int(drafts[0, 0]) + 1) % w.vocab     # not the proposer's argmax: q(draft) = 0
    mod = dict(inputs, drafts=drafts)
    gpu = helpers.run_gpu(w, mod, diag=True, dump_r=True)
    ref = helpers.run_oracle(w, mod, return_r=True)
    helpers.check_parity(w, gpu, ref, check_diag=False)
    helpers.check_combined_probabilities(w, gpu["r"], ref["r"])
    assert gpu["row_status"][0] & COS_ROW_Q_ZERO


@pytest.mark.parametrize("name", ["cfg5_greedy", "cfg2_greedy", "we_greedy"])
def test_greedy_with_non_finite_logits(name):
    """T = 0 (Sec. 4.1: one-hot distributions): a NaN or +inf among a position's logits, or a model without a
    finite maximum, leaves the argmax undefined: the position counts as rejected, no token, NONFINITE; -inf
    entries are legal while a finite maximum remains.  Rows against the oracle."""
    if name == "cfg5_greedy":
        w = C["cfg5_greedy"].scaled(batch=8, vocab=16000, gamma=3, name="greedy_nonfinite")
    elif name == "cfg2_greedy":
        w = synth.Workload("cd_greedy", 2, 1, (1.0, -0.5), 0.0, 8, 3, 9001, "bf16", "gauss", sigma=3.0, rho=0.7,
                           proposer_rule="cycle", mask_model=0, mask_alpha=0.1)
    else:
        w = synth.Workload("we_greedy_nf", 3, 0, (0.5, 0.3, 0.2), 0.0, 8, 3, 5000, "f32", "gauss", sigma=2.0, rho=0.5,
                           proposer_rule="cycle")
    inputs = synth.make_inputs(w, "cuda")
    logits = inputs["logits"].clone()
    logits[0, 0, 0, 17] = float("nan")            # row 0 stops at position 0
    logits[1, 1, 1, 3] = float("inf")             # row 1 at position 1 at the latest
    logits[w.n - 1, 2, 2, :] = float("-inf")      # a model with no finite maximum
    worst = int(torch.argmin(logits[0, 3, 0].float()))
    logits[0, 3, :, worst] = float("-inf")        # a ruled-out token that is nobody's argmax: harmless
    mod = dict(inputs, logits=logits)
    gpu = helpers.run_gpu(w, mod, diag=True)
    ref = helpers.run_oracle(w, mod)
    helpers.check_parity(w, gpu, ref, check_diag=False)
    assert gpu["accept_count"][0] == 0 and gpu["out_tokens"][0, 0] == -1 and gpu["row_status"][0] & COS_ROW_NONFINITE
    assert gpu["accept_count"][1] <= 1 and gpu["accept_count"][2] <= 2
    for b in (1, 2):
        if gpu["row_status"][b] & COS_ROW_NONFINITE:
            assert gpu["out_tokens"][b, gpu["accept_count"][b]] == -1
    assert not (gpu["row_status"][3] & COS_ROW_NONFINITE)


@pytest.mark.parametrize("name", ["cfg3", "cfg5", "cfg5_greedy"])
def test_proposer_index_outside_the_models_is_reported_per_row(name):
    """A proposer index outside [0, n) names no distribution q: every position of that row reports NONFINITE
    (so the row stops at position 0 without a token); the other rows are those of the oracle."""
    w = C[name].scaled(batch=6, vocab=8192, gamma=3, name=f"{name}_bad_proposer")
    inputs = synth.make_inputs(w, "cuda")
    prop = inputs["proposer"].clone()
    prop[1] = w.n
    prop[4] = -1
    gpu = helpers.run_gpu(w, dict(inputs, proposer=prop), diag=True)
    ref = helpers.run_oracle(w, inputs)
    good = [0, 2, 3, 5]
    helpers.check_parity(w, gpu, ref, rows=good)
    for b in (1, 4):
        assert gpu["accept_count"][b] == 0 and gpu["row_status"][b] & COS_ROW_NONFINITE
        assert np.all(gpu["out_tokens"][b] == -1)


def test_invalid_arguments_return_errors():
    w = _small("cfg3", batch=2, vocab=1024, gamma=2, name="args")
    inputs = synth.make_inputs(w, "cuda")
    v = helpers.make_verifier(w)
    try:
        with pytest.raises(CosVerifyError):        # batch larger than max_batch
            big = torch.zeros((w.n, 3, w.gamma + 1, w.vocab), dtype=inputs["logits"].dtype, device="cuda")
            v.run(big, torch.zeros((3, w.gamma), dtype=torch.int32, device="cuda"),
                  torch.zeros(3, dtype=torch.int32, device="cuda"), 1, 0)
        with pytest.raises(ValueError):            # wrong vocabulary
            v.run(inputs["logits"][..., :-8], inputs["drafts"], inputs["proposer"], 1, 0)
        with pytest.raises(CosVerifyError):        # host-pointer call without staging
            v.run_host(inputs["logits"].cpu(), inputs["drafts"].cpu(), inputs["proposer"].cpu(), 1, 0)
        with pytest.raises(CosVerifyError):        # bonus model outside [0, n)
            v.run(inputs["logits"], inputs["drafts"], inputs["proposer"], 1, 0, bonus_model=w.n)
        with pytest.raises(CosVerifyError):        # unknown flag bit
            v.run(inputs["logits"], inputs["drafts"], inputs["proposer"], 1, 0, flags=1 << 9)
        with pytest.raises(ValueError):            # a proposer table of the wrong shape
            v.run(inputs["logits"], inputs["drafts"], torch.zeros((2, w.gamma), dtype=torch.int32, device="cuda"), 1, 0)
        with pytest.raises(ValueError):            # the device-resident offset must be an int64 device tensor
            v.run(inputs["logits"], inputs["drafts"], inputs["proposer"], 1, 0,
                  offset_device=torch.zeros(1, dtype=torch.int32, device="cuda"))
        ok = v.run(inputs["logits"], inputs["drafts"], inputs["proposer"], 1, 0)   # the context still works
        torch.cuda.synchronize()
        assert ok["accept_count"].min() >= 0
    finally:
        v.close()


@pytest.mark.parametrize("name", ["cfg3", "cfg5_greedy"])
def test_early_exit_hint_gives_the_rows_of_the_full_run(name):
    """COS_RUN_EARLY_EXIT: positions behind a rejection their row has already reported may be left unread
    (Sec. 3.1 discards them).  The rows must be those of the full run; what is reported for positions up to
    and including the first rejection must be there; some later positions are in fact left unread."""
    from paper_2502_01662_b200 import COS_RUN_EARLY_EXIT
    w = C[name]
    inputs = synth.make_inputs(w, "cuda")
    v = helpers.make_verifier(w)
    try:
        full = helpers.run_gpu(w, inputs, verifier=v, diag=True)
        hint = helpers.run_gpu(w, inputs, verifier=v, diag=True, flags=COS_RUN_EARLY_EXIT)
        again = helpers.run_gpu(w, inputs, verifier=v, diag=True)        # the scratch was left clean
    finally:
        v.close()
    for k in ("accept_count", "out_tokens", "row_status"):
        assert np.array_equal(hint[k], full[k]), k
        assert np.array_equal(again[k], full[k]), k
    assert np.array_equal(np.isnan(hint["bonus_prob"]), np.isnan(full["bonus_prob"]))
    # and a sample of the hinted run's rows against the oracle itself
    rows = sorted(np.random.default_rng(13).choice(w.batch, size=24, replace=False).tolist())
    ref = helpers.run_oracle(w, inputs, rows=rows, native=True)
    helpers.check_parity(w, hint, ref, rows=rows, check_diag=False)
    a = full["accept_count"]
    g = w.gamma
    unread = 0
    for b in range(w.batch):
        for j in range(g):
            if j <= a[b]:
                assert np.array_equal(hint["diag"][b, j, :3], full["diag"][b, j, :3], equal_nan=True), (b, j)
            elif np.isnan(hint["diag"][b, j, 1]) and not np.isnan(full["diag"][b, j, 1]):
                unread += 1
    # workload 3 keeps every position resident at once, so nothing can be known in time there; workload 5
    # runs in many waves and leaves positions unread
    assert unread > 0 or name == "cfg3"
    del inputs
    torch.cuda.empty_cache()


@pytest.mark.parametrize("name,kw", [("cfg3", dict(batch=40, vocab=20008, gamma=8)), ("cfg5", dict(batch=6, vocab=50000, gamma=3)),
                                     ("cfg2", dict(batch=8, vocab=9001, gamma=5)), ("cfg5_greedy", dict(batch=6, vocab=50000, gamma=3))])
def test_a_run_can_be_captured_in_a_graph_and_replayed(name, kw):
    """The launches of a run depend on its arguments only, and the kernels leave the scratch as they found it:
    a captured run, replayed with the counter offset kept in device memory, gives what an ordinary run with
    that offset gives."""
    w = C[name].scaled(**kw)
    inputs = synth.make_inputs(w, "cuda")
    B, P = w.batch, w.gamma + 1
    v, ref_v = helpers.make_verifier(w), helpers.make_verifier(w)
    try:
        off = torch.zeros(1, dtype=torch.int64, device="cuda")
        outs = v._alloc_outs(B, P, w.vocab, torch.device("cuda"), True, False)
        args = (inputs["logits"], inputs["drafts"], inputs["proposer"], inputs["seed"], 0)
        v.run(*args, outs=outs, offset_device=off)          # an ordinary run first
        torch.cuda.synchronize()
        g = torch.cuda.CUDAGraph()
        with torch.cuda.graph(g):
            v.run(*args, outs=outs, offset_device=off)
        for k in (3, 4, 1 << 40):
            off.fill_(k)
            for t in outs.values():
                t.zero_()
            g.replay()
            torch.cuda.synchronize()
            want = ref_v.run(inputs["logits"], inputs["drafts"], inputs["proposer"], inputs["seed"], k, diag=True)
            torch.cuda.synchronize()
            for key in ("accept_count", "out_tokens", "row_status"):
                assert torch.equal(outs[key], want[key]), (k, key)
            assert torch.equal(torch.nan_to_num(outs["diag"], nan=-7.0), torch.nan_to_num(want["diag"], nan=-7.0))
            assert torch.equal(torch.nan_to_num(outs["bonus_prob"], nan=-7.0), torch.nan_to_num(want["bonus_prob"], nan=-7.0))
        # an ordinary run after the replays still works on the same context
        again = v.run(inputs["logits"], inputs["drafts"], inputs["proposer"], inputs["seed"], 3)
        want = ref_v.run(inputs["logits"], inputs["drafts"], inputs["proposer"], inputs["seed"], 3)
        torch.cuda.synchronize()
        assert torch.equal(again["out_tokens"], want["out_tokens"])
    finally:
        v.close()
        ref_v.close()


@pytest.mark.parametrize("name,kw", [("cfg3", dict(batch=40, vocab=20008, gamma=8)), ("cfg4", dict(batch=30, vocab=12808, gamma=5)),
                                     ("cfg5", dict(batch=36, vocab=16000, gamma=4)), ("cfg5_greedy", dict(batch=36, vocab=16000, gamma=4)),
                                     ("cfg2", dict(batch=8, vocab=9001, gamma=5))])
@pytest.mark.parametrize("settled", [False, True])
def test_calls_queued_back_to_back_give_what_isolated_calls_give(name, kw, settled):
    """Every launch of a run may take its places on the device while the kernel before it in the stream drains,
    and waits for that kernel before it reads or writes anything.  Sixteen calls queued without a pause, on
    logits that a kernel queued just before each call writes, into output buffers of their own, must give what
    the same calls give one by one with a synchronisation in between.  With COS_RUN_INPUTS_SETTLED (inputs that
    were complete long before: no producer kernel) the streaming launch reads them while the previous call's
    drawing launch drains, and the results are the same again."""
    w = C[name].scaled(**kw)
    inputs = synth.make_inputs(w, "cuda")
    B, P = w.batch, w.gamma + 1
    v = helpers.make_verifier(w)
    try:
        variants = [torch.roll(inputs["logits"], shifts=7 * k, dims=-1) for k in range(4)]
        drafts = [((inputs["drafts"] + 7 * k) % w.vocab).to(torch.int32) for k in range(4)]   # rolled with the logits
        live = torch.empty_like(inputs["logits"])
        queued = []
        for k in range(16):
            outs = v._alloc_outs(B, P, w.vocab, torch.device("cuda"), True, False)
            if settled:
                v.run(variants[k % 4], drafts[k % 4], inputs["proposer"], inputs["seed"], 100 + k, outs=outs,
                      flags=COS_RUN_INPUTS_SETTLED)
            else:
                live.copy_(variants[k % 4])                  # a kernel in the same stream produces the logits
                v.run(live, drafts[k % 4], inputs["proposer"], inputs["seed"], 100 + k, outs=outs)
            queued.append(outs)
        torch.cuda.synchronize()
        for k in range(16):
            want = v.run(variants[k % 4], drafts[k % 4], inputs["proposer"], inputs["seed"], 100 + k, diag=True)
            torch.cuda.synchronize()
            for key in ("accept_count", "out_tokens", "row_status"):
                assert torch.equal(queued[k][key], want[key]), (k, key)
            assert torch.equal(torch.nan_to_num(queued[k]["diag"], nan=-7.0), torch.nan_to_num(want["diag"], nan=-7.0)), k
        # and one of them against the oracle
        ref = helpers.run_oracle(w, dict(inputs, logits=variants[1], drafts=drafts[1], offset=101), native=True)
        got = {key: t.cpu().numpy() for key, t in queued[1].items()}
        helpers.check_parity(w, got, ref)
    finally:
        v.close()
