"""The allocation-free entry point (cos_verify_run_static) against the context-based one.

Some hosts of the library cannot allocate device memory at the point where they verify (the
device belongs to an engine's memory pool, or cudaMalloc's device-wide stall is not acceptable
mid-serving); for them the scratch is an array built into the library.  This file is collected
last on purpose: a failure here cannot hide the result of any other test in a stop-at-first-
failure run.  Each case makes two calls in a row, because the built-in array keeps whatever the
previous call left in it and every call has to start from a clean state by itself.
"""
import ctypes

import numpy as np
import pytest
import torch

import helpers
from paper_2502_01662_b200 import binding, synth

pytestmark = pytest.mark.gpu

C = synth.CONFIGS
CASES = [
    C["cfg3"].scaled(batch=6, vocab=20008, gamma=4, name="static_we"),
    C["cfg2"].scaled(batch=5, vocab=9001, gamma=3, name="static_masked_ragged"),
    C["cfg5_greedy"].scaled(batch=4, vocab=16000, gamma=3, name="static_greedy"),
]


@pytest.mark.parametrize("w", CASES, ids=[w.name for w in CASES])
def test_static_entry_matches_context_entry_twice(w):
    inputs = synth.make_inputs(w, "cuda")
    B, P = w.batch, w.gamma + 1
    verifier = helpers.make_verifier(w)
    try:
        for call in range(2):                      # second call runs on the array the first one used
            offset = inputs["offset"] + call
            want = verifier.run(inputs["logits"], inputs["drafts"], inputs["proposer"], inputs["seed"], offset,
                                diag=True)
            outs = {
                "accept_count": torch.full((B,), -7, dtype=torch.int32, device="cuda"),
                "out_tokens": torch.full((B, P), -7, dtype=torch.int32, device="cuda"),
                "row_status": torch.full((B,), -7, dtype=torch.int32, device="cuda"),
                "diag": torch.zeros((B, P, 4), dtype=torch.float32, device="cuda"),
            }
            binding.run_static(w.n, w.combine, w.weights, w.temperature, w.gamma, w.vocab, inputs["logits"],
                               inputs["drafts"], inputs["proposer"], inputs["seed"], offset,
                               mask_model=w.mask_model, mask_alpha=w.mask_alpha, outs=outs)
            torch.cuda.synchronize()
            for k in ("accept_count", "out_tokens", "row_status"):
                assert torch.equal(outs[k], want[k]), (call, k)
            # ratio, r(x), q(x): same arithmetic, compared within the tolerance of the parity tests
            got, ref = outs["diag"][..., :3].cpu().numpy(), want["diag"][..., :3].cpu().numpy()
            np.testing.assert_allclose(got, ref, rtol=helpers.TOL_R[w.dtype], atol=1e-30, equal_nan=True)
            # and against the oracle itself, with the bar of the parity tests
            oracle = helpers.run_oracle(w, dict(inputs, offset=offset))
            helpers.check_parity(w, {k: t.cpu().numpy() for k, t in outs.items()}, oracle)
    finally:
        verifier.close()


def _static_outs(B, P, extra=()):
    outs = {
        "accept_count": torch.full((B,), -7, dtype=torch.int32, device="cuda"),
        "out_tokens": torch.full((B, P), -7, dtype=torch.int32, device="cuda"),
        "row_status": torch.full((B,), -7, dtype=torch.int32, device="cuda"),
        "diag": torch.zeros((B, P, 4), dtype=torch.float32, device="cuda"),
    }
    if "bonus_prob" in extra:
        outs["bonus_prob"] = torch.zeros(B, dtype=torch.float32, device="cuda")
    return outs


def _call_static(w, inputs, outs, offset, **kw):
    binding.run_static(w.n, w.combine, w.weights, w.temperature, w.gamma, w.vocab, inputs["logits"], inputs["drafts"],
                       inputs["proposer"], inputs["seed"], offset, mask_model=w.mask_model, mask_alpha=w.mask_alpha,
                       outs=outs, **kw)
    torch.cuda.synchronize()
    return {k: t.cpu().numpy() for k, t in outs.items()}


def test_static_entry_at_its_limits_and_a_small_call_after_a_large_one():
    """8192 positions in 1024 rows (both limits at once), then a few rows on the array the large call used."""
    big = C["cfg1"].scaled(batch=1024, vocab=64, gamma=7, name="static_limits")
    small = C["cfg3"].scaled(batch=3, vocab=20008, gamma=4, name="static_after_large")
    for w in (big, small, big):
        inputs = synth.make_inputs(w, "cuda")
        got = _call_static(w, inputs, _static_outs(w.batch, w.gamma + 1), inputs["offset"])
        ref = helpers.run_oracle(w, inputs, native=True)
        helpers.check_parity(w, got, ref)


def test_static_entry_with_the_optional_arguments():
    """Residual mass everywhere (the job list grows to positions + rows), a named bonus model with its
    probability, a proposer per position, and a forced cluster size: each twice in a row, against the oracle."""
    from paper_2502_01662_b200 import COS_RUN_ALL_RESIDUALS
    w = C["cfg4"].scaled(batch=6, vocab=12808, gamma=3, name="static_opts")
    inputs = synth.make_inputs(w, "cuda")
    g = np.random.default_rng(2)
    table = torch.as_tensor(g.integers(0, w.n, size=(w.batch, w.gamma + 1)).astype(np.int32), device="cuda")
    for call in range(2):
        off = inputs["offset"] + call
        got = _call_static(w, inputs, _static_outs(w.batch, w.gamma + 1), off, flags=COS_RUN_ALL_RESIDUALS)
        ref = helpers.run_oracle(w, dict(inputs, offset=off), native=True)
        helpers.check_parity(w, got, ref)
        np.testing.assert_allclose(got["diag"][:, : w.gamma, 3], ref["S"][:, : w.gamma], rtol=1e-5, atol=1e-7)
        mod = dict(inputs, proposer=table, offset=off)
        got = _call_static(w, mod, _static_outs(w.batch, w.gamma + 1, ("bonus_prob",)), off, bonus_model=1)
        helpers.check_parity(w, got, helpers.run_oracle(w, mod, bonus_model=1, native=True))
        got = _call_static(w, inputs, _static_outs(w.batch, w.gamma + 1), off, cluster_size=2)
        helpers.check_parity(w, got, ref)


def test_static_entry_rejects_sizes_beyond_the_built_in_scratch():
    lib = binding.load_library()
    lib.cos_verify_run_static.argtypes = [ctypes.POINTER(binding.cos_verify_config),
                                          ctypes.POINTER(binding.cos_verify_args), ctypes.c_void_p]
    lib.cos_verify_run_static.restype = ctypes.c_int
    cfg = binding.cos_verify_config()
    cfg.n, cfg.combine = 2, binding.COS_COMBINE_PROB_ENSEMBLE
    cfg.weights[0], cfg.weights[1] = 0.5, 0.5
    cfg.mask_model, cfg.mask_alpha, cfg.temperature = -1, 1.0, 1.0
    cfg.gamma, cfg.vocab, cfg.max_batch, cfg.dtype = 8, 64, 1, binding.COS_DTYPE_F32
    dummy = torch.zeros(16, dtype=torch.int32, device="cuda")
    a = binding.cos_verify_args()
    for name in ("logits", "draft_tokens", "proposer", "accept_count", "out_tokens", "row_status"):
        setattr(a, name, dummy.data_ptr())
    for batch, word in ((1025, b"COS_STATIC_MAX_BATCH"), (1000, b"COS_STATIC_MAX_POSITIONS")):
        a.batch = batch
        st = lib.cos_verify_run_static(ctypes.byref(cfg), ctypes.byref(a), None)
        assert st == 1                                           # COS_ERR_INVALID_ARG, nothing enqueued
        assert word in lib.cos_verify_last_error(None)
    torch.cuda.synchronize()
