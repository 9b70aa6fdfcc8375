"""Seeded synthetic workloads: logits, draft tokens and proposer indices.

These stand in for the model pairs and datasets of the paper's experiments (Sec. 4.1,
Table 1), keeping their shapes: vocabularies of 32000 (Llama-2 / Vicuna), 128256
(Llama-3), 151936 (Qwen2.5) and a 256000 stress case; two to four models; proposal
lengths around the paper's gamma = 5.  This module only produces inputs: it contains
none of the verification arithmetic, and both the CUDA path and the test oracle read the
bytes it returns.

Generators (every tensor follows from `seed`):
  gauss        l_i = sigma * (sqrt(rho) z + sqrt(1-rho) e_i),  z, e_i ~ N(0,1), z shared by the models
  gumbel_zipf  l_i = 3 * (sqrt(rho) g + sqrt(1-rho) e_i) - 1.1 ln(rank(x)),  g, e_i standard Gumbel,
               rank = one seeded permutation of the tokens shared by all models and rows
Values are rounded once to the storage dtype.  Draft tokens are drawn from the proposer's
tempered softmax by float64 inverse CDF with uniforms from numpy's Philox generator
(argmax at T = 0).
"""
from __future__ import annotations

import math
from dataclasses import dataclass, replace
from typing import Dict, Optional, Sequence

import numpy as np
import torch

COMBINE_PROB_ENSEMBLE = 0
COMBINE_LOGIT_LINEAR = 1


@dataclass(frozen=True)
class Workload:
    name: str
    n: int
    combine: int
    weights: Sequence[float]
    temperature: float
    batch: int
    gamma: int
    vocab: int
    dtype: str                  # "f32", "bf16" or "f16"
    generator: str              # "gauss" or "gumbel_zipf"
    sigma: float = 1.0          # gauss only
    rho: float = 0.8
    proposer_rule: str = "zero"  # "zero", "cycle" (b mod n) or "bernoulli"
    mask_model: int = -1
    mask_alpha: float = 1.0
    seed: int = 20250201
    verify_seed: int = 0x5EEDC05C05
    verify_offset: int = 0

    @property
    def positions(self) -> int:
        return self.batch * (self.gamma + 1)

    @property
    def elem_bytes(self) -> int:
        return 4 if self.dtype == "f32" else 2

    @property
    def bytes_per_position(self) -> int:
        """Algorithmic bytes: every logit of every model is read once."""
        return self.n * self.vocab * self.elem_bytes

    @property
    def torch_dtype(self):
        return {"bf16": torch.bfloat16, "f16": torch.float16}.get(self.dtype, torch.float32)

    def scaled(self, batch: Optional[int] = None, vocab: Optional[int] = None, gamma: Optional[int] = None,
               name: Optional[str] = None) -> "Workload":
        """The same recipe at another size (used by the tests)."""
        return replace(self, batch=self.batch if batch is None else batch,
                       vocab=self.vocab if vocab is None else vocab,
                       gamma=self.gamma if gamma is None else gamma,
                       name=name or (self.name + "_scaled"))


CONFIGS: Dict[str, Workload] = {
    # 1: two-model ensemble, fp32, one row (a latency case)
    "cfg1": Workload("cfg1", 2, COMBINE_PROB_ENSEMBLE, (0.5, 0.5), 1.0, 1, 4, 32000, "f32", "gauss",
                     sigma=2.0, rho=0.8, proposer_rule="zero"),
    # 2: contrastive decoding with plausibility mask, expert = model 0
    "cfg2": Workload("cfg2", 2, COMBINE_LOGIT_LINEAR, (1.0, -0.5), 1.0, 8, 5, 32000, "bf16", "gauss",
                     sigma=3.0, rho=0.7, proposer_rule="cycle", mask_model=0, mask_alpha=0.1),
    # 3: two-model ensemble at T = 0.7, Qwen-sized vocabulary
    "cfg3": Workload("cfg3", 2, COMBINE_PROB_ENSEMBLE, (0.5, 0.5), 0.7, 64, 8, 151936, "bf16", "gumbel_zipf",
                     rho=0.85, proposer_rule="bernoulli"),
    # 4: four-model ensemble, proposer cycling through the models
    "cfg4": Workload("cfg4", 4, COMBINE_PROB_ENSEMBLE, (0.4, 0.3, 0.2, 0.1), 1.0, 32, 6, 128256, "bf16", "gauss",
                     sigma=2.5, rho=0.8, proposer_rule="cycle"),
    # 5: logit interpolation 1.5 * aligned - 0.5 * base, sampling and greedy
    "cfg5": Workload("cfg5", 2, COMBINE_LOGIT_LINEAR, (1.5, -0.5), 1.0, 256, 8, 256000, "bf16", "gumbel_zipf",
                     rho=0.9, proposer_rule="zero"),
    # workload 3 with the logits stored as IEEE half (a variant beside the five workloads the benchmark reports)
    "cfg3_f16": Workload("cfg3_f16", 2, COMBINE_PROB_ENSEMBLE, (0.5, 0.5), 0.7, 64, 8, 151936, "f16", "gumbel_zipf",
                         rho=0.85, proposer_rule="bernoulli"),
    "cfg5_greedy": Workload("cfg5_greedy", 2, COMBINE_LOGIT_LINEAR, (1.5, -0.5), 0.0, 256, 8, 256000, "bf16",
                            "gumbel_zipf", rho=0.9, proposer_rule="zero"),
}


def _standard_gumbel(shape, gen, device):
    e = torch.empty(shape, dtype=torch.float32, device=device).exponential_(1.0, generator=gen)
    return -torch.log(e)


def make_proposer(w: Workload) -> np.ndarray:
    if w.proposer_rule == "zero":
        return np.zeros(w.batch, dtype=np.int32)
    if w.proposer_rule == "cycle":
        return (np.arange(w.batch) % w.n).astype(np.int32)
    if w.proposer_rule == "bernoulli":
        g = np.random.Generator(np.random.Philox(key=w.seed + 7))
        return (g.random(w.batch) < 0.5).astype(np.int32)
    raise ValueError(w.proposer_rule)


def make_logits(w: Workload, device="cpu", rows_per_chunk: int = 16) -> torch.Tensor:
    """[n, B, gamma+1, V] logits in the storage dtype on `device`."""
    P, V, n, B = w.gamma + 1, w.vocab, w.n, w.batch
    dev = torch.device(device)
    gen = torch.Generator(device=dev)
    gen.manual_seed(w.seed)
    out = torch.empty((n, B, P, V), dtype=w.torch_dtype, device=dev)
    if w.generator == "gumbel_zipf":
        perm = torch.randperm(V, generator=gen, device=dev)
        rank = torch.empty(V, dtype=torch.float32, device=dev)
        rank[perm] = torch.arange(1, V + 1, dtype=torch.float32, device=dev)
        bias = -1.1 * torch.log(rank)
    a, c = math.sqrt(w.rho), math.sqrt(1.0 - w.rho)
    for b0 in range(0, B, rows_per_chunk):
        b1 = min(B, b0 + rows_per_chunk)
        shape = (b1 - b0, P, V)
        if w.generator == "gauss":
            shared = torch.randn(shape, generator=gen, device=dev)
            for i in range(n):
                own = torch.randn(shape, generator=gen, device=dev)
                out[i, b0:b1] = (w.sigma * (a * shared + c * own)).to(w.torch_dtype)
        elif w.generator == "gumbel_zipf":
            shared = _standard_gumbel(shape, gen, dev)
            for i in range(n):
                own = _standard_gumbel(shape, gen, dev)
                out[i, b0:b1] = (3.0 * (a * shared + c * own) + bias).to(w.torch_dtype)
        else:
            raise ValueError(w.generator)
    return out


def make_drafts(w: Workload, logits: torch.Tensor, proposer: np.ndarray, rows_per_chunk: int = 16) -> np.ndarray:
    """[B, gamma] draft tokens drawn from the proposer's softmax at temperature T."""
    B, g, V = w.batch, w.gamma, w.vocab
    drafts = np.zeros((B, g), dtype=np.int32)
    if g == 0:
        return drafts
    u = np.random.Generator(np.random.Philox(key=w.seed + 13)).random((B, g))
    prop = torch.as_tensor(proposer.astype(np.int64), device=logits.device)
    for b0 in range(0, B, rows_per_chunk):
        b1 = min(B, b0 + rows_per_chunk)
        idx = prop[b0:b1]
        rows = logits[idx, torch.arange(b0, b1, device=logits.device), :g, :].to(torch.float64)   # [rows, g, V]
        if w.temperature == 0.0:
            tok = torch.argmax(rows, dim=-1)
        else:
            cdf = torch.cumsum(torch.softmax(rows / w.temperature, dim=-1), dim=-1)
            uu = torch.as_tensor(u[b0:b1], device=logits.device).unsqueeze(-1) * cdf[..., -1:]
            tok = torch.searchsorted(cdf, uu).squeeze(-1).clamp_(max=V - 1)
        drafts[b0:b1] = tok.cpu().numpy().astype(np.int32)
    return drafts


def make_inputs(w: Workload, device="cpu") -> dict:
    """All inputs of one verification call for workload `w`."""
    logits = make_logits(w, device)
    proposer = make_proposer(w)
    drafts = make_drafts(w, logits, proposer)
    return {
        "logits": logits,
        "drafts": torch.as_tensor(drafts, device=logits.device),
        "proposer": torch.as_tensor(proposer, device=logits.device),
        "seed": w.verify_seed,
        "offset": w.verify_offset,
    }


def logits_as_numpy(logits: torch.Tensor) -> np.ndarray:
    """Host copy for a CPU consumer: float32 or float16 array, or the raw 16-bit patterns of bf16."""
    t = logits.detach().cpu().contiguous()
    if t.dtype == torch.bfloat16:
        return t.view(torch.int16).numpy().view(np.uint16)
    return t.numpy()
