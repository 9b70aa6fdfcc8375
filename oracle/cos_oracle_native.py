"""ctypes front of cos_oracle.cpp, the C++ twin of the float64 oracle (TEST INFRASTRUCTURE, not product code).

Same arguments and the same result dictionary as cos_oracle.verify, so tests can run either; the C++ one spreads
the rows over host threads (OpenMP), which makes full-size workloads checkable on every row.  It is compiled
here with g++ on first use; nothing under paper_2502_01662_b200/ loads it.
"""
from __future__ import annotations

import ctypes
import os
import subprocess
from typing import Optional, Sequence

import numpy as np

_DIR = os.path.dirname(os.path.abspath(__file__))
SRC = os.path.join(_DIR, "cos_oracle.cpp")
LIB = os.path.join(_DIR, "libcos_oracle.so")
_lib = None


def build(force: bool = False) -> str:
    """Plain g++ -O2 with OpenMP, floating-point contraction off, no fast-math."""
    if force or not os.path.exists(LIB) or os.path.getmtime(LIB) < os.path.getmtime(SRC):
        cmd = ["g++", "-O2", "-std=c++17", "-fopenmp", "-ffp-contract=off", "-fPIC", "-shared", "-o", LIB, SRC]
        res = subprocess.run(cmd, capture_output=True, text=True)
        if res.returncode != 0:
            raise RuntimeError("g++ failed:\n" + " ".join(cmd) + "\n" + res.stderr)
    return LIB


def load():
    global _lib
    if _lib is None:
        _lib = ctypes.CDLL(build())
        _lib.cos_oracle_max_threads.restype = ctypes.c_int
        _lib.cos_oracle_verify.restype = ctypes.c_int
    return _lib


def max_threads() -> int:
    return int(load().cos_oracle_max_threads())


def _ptr(a):
    return a.ctypes.data_as(ctypes.c_void_p) if a is not None else None


def verify(logits, dtype: str, drafts, proposer, cfg, seed: int, offset: int, row_base: int = 0,
           rows: Optional[Sequence[int]] = None, threads: int = 0) -> dict:
    """cos_oracle.verify in C++: logits [n, B, gamma+1, V] (uint16 patterns for 'bf16', float16 for 'f16',
    float32 for 'f32'), `cfg` an OracleConfig.  `threads` = 0 lets OpenMP choose."""
    lib = load()
    logits = np.ascontiguousarray(logits)
    n, B, P, V = logits.shape
    g = cfg.gamma
    assert P == g + 1 and n == cfg.n and V == cfg.vocab
    code = {"f32": 0, "bf16": 1, "f16": 2}[dtype]
    if dtype == "bf16" and logits.dtype != np.uint16:
        logits = logits.view(np.uint16)
    if dtype == "f16":
        logits = logits.view(np.uint16)
    if dtype == "f32":
        logits = logits.astype(np.float32, copy=False)
    drafts = np.ascontiguousarray(np.asarray(drafts, dtype=np.int32).reshape(B, g)) if g > 0 else np.zeros((B, 0), np.int32)
    proposer = np.ascontiguousarray(np.asarray(proposer, dtype=np.int32))
    per_pos = 0 if (proposer.size == B and proposer.ndim <= 1) else 1
    weights = np.zeros(8, np.float32)
    weights[: cfg.n] = np.asarray(cfg.weights, dtype=np.float32)[: cfg.n]
    rows_arr = None if rows is None else np.ascontiguousarray(np.asarray(list(rows), dtype=np.int32))
    out = {
        "accept_count": np.full(B, -1, np.int32), "out_tokens": np.full((B, P), -1, np.int32),
        "row_status": np.zeros(B, np.uint32), "bonus_prob": np.full(B, np.nan),
        "accept": np.zeros((B, P), np.uint8), "cand": np.full((B, P), -1, np.int64),
        "ratio": np.full((B, P), np.nan), "r_d": np.full((B, P), np.nan), "q_d": np.full((B, P), np.nan),
        "S": np.full((B, P), np.nan), "boundary_accept": np.zeros((B, P), np.uint8),
        "boundary_sample": np.zeros((B, P), np.uint8), "pos_status": np.zeros((B, P), np.uint32),
        "u_acc": np.zeros((B, P)), "u_smp": np.zeros((B, P)),
    }
    s = [st // logits.itemsize for st in logits.strides]
    rc = lib.cos_oracle_verify(
        _ptr(logits), ctypes.c_int(code), ctypes.c_longlong(s[0]), ctypes.c_longlong(s[1]), ctypes.c_longlong(s[2]),
        ctypes.c_int(n), ctypes.c_int(B), ctypes.c_int(g), ctypes.c_int(V), ctypes.c_int(cfg.combine), _ptr(weights),
        ctypes.c_float(cfg.temperature), ctypes.c_int(cfg.mask_model), ctypes.c_float(cfg.mask_alpha),
        ctypes.c_int(cfg.bonus_model), _ptr(drafts), _ptr(proposer), ctypes.c_int(per_pos),
        ctypes.c_ulonglong(seed & 0xFFFFFFFFFFFFFFFF), ctypes.c_ulonglong(offset & 0xFFFFFFFFFFFFFFFF),
        ctypes.c_longlong(row_base), _ptr(rows_arr), ctypes.c_int(0 if rows_arr is None else len(rows_arr)),
        ctypes.c_int(threads), _ptr(out["accept_count"]), _ptr(out["out_tokens"]), _ptr(out["row_status"]),
        _ptr(out["bonus_prob"]), _ptr(out["accept"]), _ptr(out["cand"]), _ptr(out["ratio"]), _ptr(out["r_d"]),
        _ptr(out["q_d"]), _ptr(out["S"]), _ptr(out["boundary_accept"]), _ptr(out["boundary_sample"]),
        _ptr(out["pos_status"]), _ptr(out["u_acc"]), _ptr(out["u_smp"]))
    if rc != 0:
        raise ValueError("cos_oracle_verify rejected its arguments")
    for k in ("accept", "boundary_accept", "boundary_sample"):
        out[k] = out[k].astype(bool)
    return out
