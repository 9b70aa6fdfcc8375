"""Shared plumbing of the GPU parity tests: run both sides on the same inputs and compare.

Bit-exact bar: accept counts, emitted tokens and row status must be identical, except for
rows whose first difference sits at a position the oracle marks as a boundary case
(|u - min(1, ratio)| < 1e-5 for the accept test, a normalised CDF edge within 1e-6 of u
for the sample).  Those rows are counted and reported, never silently dropped.
"""
from __future__ import annotations

import numpy as np

from oracle import cos_oracle as orc
from paper_2502_01662_b200 import synth

TOL_R = {"f32": 1e-5, "bf16": 2e-3, "f16": 2e-3}      # relative tolerance on combined probabilities
FLOOR_R = 1e-30                          # fp32 cannot hold probabilities far below this


def oracle_config(w: synth.Workload, bonus_model: int = -1) -> orc.OracleConfig:
    return orc.OracleConfig(n=w.n, combine=w.combine, weights=list(w.weights), temperature=w.temperature,
                            gamma=w.gamma, vocab=w.vocab, mask_model=w.mask_model, mask_alpha=w.mask_alpha,
                            bonus_model=bonus_model)


def run_oracle(w: synth.Workload, inputs: dict, rows=None, return_r=False, row_base=0, bonus_model: int = -1,
               native: bool = False, threads: int = 0) -> dict:
    """The oracle on the inputs of a GPU run.  `native` runs its C++ twin (same rows, spread over host threads),
    which is how full-size workloads are checked on every row."""
    logits = inputs["logits"]
    if native:
        from oracle import cos_oracle_native as nat
        assert not return_r
        return nat.verify(synth.logits_as_numpy(logits), w.dtype, inputs["drafts"].cpu().numpy(),
                          inputs["proposer"].cpu().numpy(), oracle_config(w, bonus_model), inputs["seed"], inputs["offset"],
                          row_base=row_base, rows=rows, threads=threads)
    if rows is not None:
        # copy only the sampled rows to the host (full-size cases hold gigabytes)
        sel = logits[:, list(rows)]
        host = synth.logits_as_numpy(sel)
        full = np.zeros((w.n, w.batch) + host.shape[2:], dtype=host.dtype)
        full[:, list(rows)] = host
        host = full
    else:
        host = synth.logits_as_numpy(logits)
    return orc.verify(host, w.dtype, inputs["drafts"].cpu().numpy(), inputs["proposer"].cpu().numpy(),
                      oracle_config(w, bonus_model), inputs["seed"], inputs["offset"], row_base=row_base, rows=rows,
                      return_r=return_r)


def make_verifier(w: synth.Workload, max_batch=None, **kw):
    from paper_2502_01662_b200 import CosVerifier
    return CosVerifier(w.n, w.combine, w.weights, w.temperature, w.gamma, w.vocab, max_batch or w.batch,
                       w.torch_dtype, mask_model=w.mask_model, mask_alpha=w.mask_alpha, **kw)


def run_gpu(w: synth.Workload, inputs: dict, verifier=None, **kw) -> dict:
    import torch
    own = verifier is None
    v = make_verifier(w) if own else verifier
    try:
        outs = v.run(inputs["logits"], inputs["drafts"], inputs["proposer"], inputs["seed"], inputs["offset"], **kw)
        torch.cuda.synchronize()
        return {k: t.cpu().numpy() for k, t in outs.items()}
    finally:
        if own:
            v.close()


def check_parity(w: synth.Workload, gpu: dict, ref: dict, rows=None, check_diag=True) -> dict:
    """Assert the bit-exact bar and return the counts of disclosed boundary rows."""
    rows = range(w.batch) if rows is None else rows
    g = w.gamma
    excused_accept = excused_sample = 0
    for b in rows:
        a_g, a_o = int(gpu["accept_count"][b]), int(ref["accept_count"][b])
        t_g, t_o = gpu["out_tokens"][b], ref["out_tokens"][b]
        if a_g == a_o and np.array_equal(t_g, t_o):
            assert int(gpu["row_status"][b]) == int(ref["row_status"][b]), (b, gpu["row_status"][b], ref["row_status"][b])
            continue
        if a_g != a_o:
            j = min(a_g, a_o)
            assert 0 <= j < g and ref["boundary_accept"][b, j], \
                f"row {b}: accept_count {a_g} vs oracle {a_o}, position {j} is not a boundary case " \
                f"(u={ref['u_acc'][b, j]!r}, ratio={ref['ratio'][b, j]!r})"
            # up to the boundary position the two rows agree, and the kernel's own ratio is the oracle's
            assert np.array_equal(t_g[:j], t_o[:j]), (b, t_g, t_o)
            if check_diag and "diag" in gpu and np.isfinite(ref["ratio"][b, j]):
                assert abs(gpu["diag"][b, j, 0] - ref["ratio"][b, j]) <= 2 * TOL_R[w.dtype] * abs(ref["ratio"][b, j]) + 1e-30
            excused_accept += 1
        else:
            assert np.array_equal(t_g[:a_o], t_o[:a_o]) and np.all(t_g[a_o + 1:] == -1), (b, t_g, t_o)
            assert ref["boundary_sample"][b, a_o], \
                f"row {b}: token {t_g[a_o]} vs oracle {t_o[a_o]} at position {a_o} is not a boundary case"
            excused_sample += 1
    if check_diag and "diag" in gpu:
        tol = TOL_R[w.dtype]
        for b in rows:
            for j in range(g):
                if ref["pos_status"][b, j] & (orc.STATUS_NONFINITE | orc.STATUS_BAD_DRAFT):
                    continue
                for k, name in ((1, "r_d"), (2, "q_d")):
                    want, got = ref[name][b, j], gpu["diag"][b, j, k]
                    assert abs(got - want) <= tol * abs(want) + FLOOR_R, (b, j, name, got, want)
                want, got = ref["ratio"][b, j], gpu["diag"][b, j, 0]
                if np.isfinite(want) and ref["q_d"][b, j] > 1e-30:
                    assert abs(got - want) <= 2 * tol * abs(want) + 1e-30, (b, j, "ratio", got, want)
                s_got = gpu["diag"][b, j, 3]
                if np.isfinite(s_got):
                    assert abs(s_got - ref["S"][b, j]) <= 1e-5 * max(ref["S"][b, j], 1e-3) + 1e-7, \
                        (b, j, "S", s_got, ref["S"][b, j])
    if "bonus_prob" in gpu and "bonus_prob" in ref:
        # probability of the bonus token under the law it was drawn from; NaN unless every draft passed
        tol = TOL_R[w.dtype]
        for b in rows:
            if int(gpu["accept_count"][b]) != int(ref["accept_count"][b]) or \
                    not np.array_equal(gpu["out_tokens"][b], ref["out_tokens"][b]):
                continue  # an excused boundary row
            want, got = ref["bonus_prob"][b], gpu["bonus_prob"][b]
            if np.isnan(want):
                assert np.isnan(got), (b, "bonus_prob", got)
            else:
                assert abs(got - want) <= tol * abs(want) + FLOOR_R, (b, "bonus_prob", got, want)
    # disclosed boundary rows are rare by construction (a band of 2e-5 per accept test, 2e-6 per sample)
    nrows = len(list(rows))
    assert excused_accept + excused_sample <= 2 + nrows * (g + 1) // 2000, (excused_accept, excused_sample, nrows)
    return {"rows": nrows, "excused_accept": excused_accept, "excused_sample": excused_sample}


def check_combined_probabilities(w: synth.Workload, r_gpu: np.ndarray, r_ref: np.ndarray, rows=None):
    rows = range(w.batch) if rows is None else rows
    tol = TOL_R[w.dtype]
    for b in rows:
        want, got = r_ref[b], r_gpu[b]
        if np.all(np.isnan(want)):
            continue
        err = np.abs(got - want)
        ok = err <= tol * np.abs(want) + FLOOR_R
        assert np.all(ok), (b, np.argwhere(~ok)[:5], got[~ok][:5], want[~ok][:5])
