"""Float64 CPU oracle for the CoS verification step (TEST INFRASTRUCTURE, not product code).

This module is the plain, slow, obviously-correct definition that the CUDA path is
checked against.  It is written from the paper alone, uses numpy in IEEE double, and
shares no code with the CUDA library.  Only tests, the smoke check and the CPU-baseline
leg of the benchmark may import it; the product never does.

What it computes, with the passage each part follows
----------------------------------------------------
* per-model distributions p_i = softmax(l_i / T)            -- Sec. 3.1 ("distributions" q_i, p_i)
* weighted ensemble      r = sum_i w_i p_i                    -- Eq. 4 (two models), n models in Sec. 4.1 / Alg. 2
* logit-level combine    r = softmax_M((sum_i w_i l_i) / T)   -- Eq. 5 (contrastive: weights (1, -mu));
                                                                 the plausibility mask M and the realignment
                                                                 weights are readings of this build, not of Eq. 5
* accept test            u <= min(1, r(x)/q(x))               -- Eq. 6 (Eq. 2 with p -> r)
* residual resample      x ~ norm(max(0, r - q))              -- Sec. 3.2, text after Eq. 6; App. A.1
* bonus token when every draft is accepted                    -- Sec. 3.1 (last sentences)
* first rejection discards the tail                           -- Sec. 3.1; Alg. 1 (reject branch)
* greedy decoding T = 0 gives one-hot distributions           -- Sec. 4.1

What the paper does not fix and this file pins as a convention ("parity unpinned" by the
paper; pinned here only by the output-law and closed-form tests):
* the coupling between uniforms and tokens: Philox4x32-10 words, u = (2*(w>>9)+1)*2^-24,
  index-order inverse CDF "smallest k with CDF_k >= u*S";
* the bonus token is drawn from the combined r at position gamma.

Every other function is pinned by tests/test_oracle_*.py (exact output law on V <= 8,
chi-squared at V = 64, closed forms, library softmax, the cuRAND host generator for the
Philox words).
"""
from __future__ import annotations

import math
from dataclasses import dataclass, field
from typing import Optional, Sequence

import numpy as np

# ----------------------------------------------------------------------------------------
# constants of the interface (values mirror the public enum meanings, not shared code)
# ----------------------------------------------------------------------------------------
COMBINE_PROB_ENSEMBLE = 0   # Eq. 4
COMBINE_LOGIT_LINEAR = 1    # Eq. 5 / logit interpolation

STATUS_NONFINITE = 1        # some distribution at a position of the row was not finite
STATUS_BAD_DRAFT = 2        # a draft token outside [0, V)
STATUS_Q_ZERO = 4           # q(draft) == 0 at some position
STATUS_RESIDUAL_EMPTY = 8   # a rejection was decided but max(0, r - q) had no mass

BOUNDARY_RATIO = 1e-5       # |u - min(1, ratio)| below this: disclosed accept boundary
BOUNDARY_CDF = 1e-6         # normalised CDF edge within this of u: disclosed sample boundary


# ----------------------------------------------------------------------------------------
# Philox4x32-10 (Salmon, Moraes, Dror, Shaw: "Parallel random numbers: as easy as 1, 2, 3",
# SC'11, Sec. 3.3 and Table 2 constants).  Vectorised over arrays of counters.
# ----------------------------------------------------------------------------------------
_PHILOX_M0 = np.uint64(0xD2511F53)
_PHILOX_M1 = np.uint64(0xCD9E8D57)
_PHILOX_W0 = 0x9E3779B9
_PHILOX_W1 = 0xBB67AE85
_MASK32 = np.uint64(0xFFFFFFFF)


def philox4x32_10(c0, c1, c2, c3, k0: int, k1: int):
    """Ten rounds of the Philox-4x32 bijection on counters (c0..c3) with key (k0, k1).

    Each round: (hi0, lo0) = M0 * c0, (hi1, lo1) = M1 * c2 (full 64-bit products), then
    c <- (hi1 ^ c1 ^ k0, lo1, hi0 ^ c3 ^ k1, lo0); the key is bumped by the Weyl
    constants between rounds.  Returns four uint32 arrays.
    """
    c0 = np.asarray(c0, dtype=np.uint64) & _MASK32
    c1 = np.asarray(c1, dtype=np.uint64) & _MASK32
    c2 = np.asarray(c2, dtype=np.uint64) & _MASK32
    c3 = np.asarray(c3, dtype=np.uint64) & _MASK32
    k0 = int(k0) & 0xFFFFFFFF
    k1 = int(k1) & 0xFFFFFFFF
    for rnd in range(10):
        if rnd > 0:
            k0 = (k0 + _PHILOX_W0) & 0xFFFFFFFF
            k1 = (k1 + _PHILOX_W1) & 0xFFFFFFFF
        p0 = _PHILOX_M0 * c0          # < 2^64, no overflow
        p1 = _PHILOX_M1 * c2
        hi0, lo0 = p0 >> np.uint64(32), p0 & _MASK32
        hi1, lo1 = p1 >> np.uint64(32), p1 & _MASK32
        c0, c1, c2, c3 = (hi1 ^ c1 ^ np.uint64(k0)), lo1, (hi0 ^ c3 ^ np.uint64(k1)), lo0
    return (c0.astype(np.uint32), c1.astype(np.uint32), c2.astype(np.uint32), c3.astype(np.uint32))


def word_to_uniform(w):
    """Map a 32-bit word to u in (0, 1): the odd multiples of 2^-24 (exact in fp32 and fp64).

    The paper only says u ~ U(0, 1) and accepts on "<=" (Eq. 2, Eq. 6); the open interval
    means ratio 0 always rejects and ratio >= 1 always accepts.
    """
    w = np.asarray(w, dtype=np.uint32)
    return (2.0 * (w >> np.uint32(9)).astype(np.float64) + 1.0) * (2.0 ** -24)


def position_uniforms(seed: int, offset: int, rows: int, positions: int, row_base: int = 0):
    """The two uniforms of every (row, position): word 0 feeds the accept test, word 1 the
    residual / bonus sample.  counter = (row_base + b, j, offset_lo, offset_hi),
    key = (seed_lo, seed_hi), so a result does not depend on how rows are batched or sharded.
    """
    b = (np.arange(rows, dtype=np.uint64) + np.uint64(row_base))[:, None] + np.zeros((1, positions), np.uint64)
    j = np.arange(positions, dtype=np.uint64)[None, :] + np.zeros((rows, 1), np.uint64)
    off_lo = np.full_like(b, offset & 0xFFFFFFFF)
    off_hi = np.full_like(b, (offset >> 32) & 0xFFFFFFFF)
    w0, w1, _, _ = philox4x32_10(b, j, off_lo, off_hi, seed & 0xFFFFFFFF, (seed >> 32) & 0xFFFFFFFF)
    return word_to_uniform(w0), word_to_uniform(w1)


# ----------------------------------------------------------------------------------------
# configuration
# ----------------------------------------------------------------------------------------
@dataclass
class OracleConfig:
    n: int
    combine: int
    weights: Sequence[float]          # stored as fp32 values, upcast exactly
    temperature: float                # fp32 value, upcast exactly; 0 = greedy
    gamma: int
    vocab: int
    mask_model: int = -1              # logit-linear only; -1 = no plausibility mask
    mask_alpha: float = 1.0           # keep x with l_e(x) >= max l_e + ln(alpha)
    bonus_model: int = -1             # -1: the token after gamma acceptances follows the combined r;
                                      # i >= 0: it follows model i's own distribution (Sec. 3.3: the
                                      # verifier's bonus token, later treated as that model's proposal)
    w64: np.ndarray = field(init=False, repr=False)

    def __post_init__(self):
        self.w64 = np.asarray(np.asarray(self.weights, dtype=np.float32)[: self.n], dtype=np.float64)
        self.temperature = float(np.float32(self.temperature))
        self.mask_alpha = float(np.float32(self.mask_alpha))
        if len(self.w64) != self.n:
            raise ValueError("need n weights")
        if not (-1 <= self.bonus_model < self.n):
            raise ValueError("bonus_model must be -1 or a model index")
        if self.combine == COMBINE_PROB_ENSEMBLE:
            if self.mask_model >= 0:
                raise ValueError("mask only with the logit-level combine")
            if np.any(self.w64 < 0) or abs(self.w64.sum() - 1.0) > 1e-6:
                raise ValueError("ensemble weights must be >= 0 and sum to 1")


def to_float64(a, dtype: str) -> np.ndarray:
    """Exact upcast of stored logits.  dtype 'bf16' means `a` holds the raw 16-bit patterns."""
    if dtype == "bf16":
        bits = np.ascontiguousarray(a).view(np.uint16) if a.dtype != np.uint16 else a
        return (bits.astype(np.uint32) << np.uint32(16)).view(np.float32).astype(np.float64)
    if dtype == "f32":
        return np.asarray(a, dtype=np.float32).astype(np.float64)
    if dtype == "f16":
        a = np.asarray(a)
        if a.dtype != np.float16:
            raise ValueError("f16 logits must be passed as a float16 array")
        return a.astype(np.float64)
    if dtype == "f64":
        return np.asarray(a, dtype=np.float64)
    raise ValueError(dtype)


# ----------------------------------------------------------------------------------------
# distributions at one position
# ----------------------------------------------------------------------------------------
def _first_argmax(v: np.ndarray) -> int:
    return int(np.argmax(v))          # numpy returns the first occurrence of the maximum


def softmax_T(l: np.ndarray, T: float) -> np.ndarray:
    """softmax(l / T) in float64 with the usual max shift (T > 0)."""
    z = l / T
    m = np.max(z)
    e = np.exp(z - m)
    return e / np.sum(e)


def plausibility_mask(l_e: np.ndarray, alpha: float) -> np.ndarray:
    """M = {x : l_e(x) >= max l_e + ln(alpha)}: tokens whose expert probability (at T = 1)
    is at least alpha times the expert's largest probability."""
    return l_e >= (np.max(l_e) + math.log(alpha))


def position_distributions(l: np.ndarray, cfg: OracleConfig, proposer: int):
    """l: [n, V] float64 logits of one (row, position).  Returns (r, q, finite_ok).

    T > 0: Eq. 4 or Eq. 5 with tempered softmaxes.  T == 0: one-hot at the lowest-index
    argmax (Sec. 4.1), the ensemble becoming a mixture of at most n atoms.
    """
    n, V = l.shape
    T = cfg.temperature
    w = cfg.w64
    with np.errstate(all="ignore"):
        if T > 0.0:
            if cfg.combine == COMBINE_PROB_ENSEMBLE:
                r = np.zeros(V, dtype=np.float64)
                q = None
                for i in range(n):
                    p_i = softmax_T(l[i], T)
                    r = r + w[i] * p_i
                    if i == proposer:
                        q = p_i
            else:
                c = np.zeros(V, dtype=np.float64)
                for i in range(n):
                    c = c + w[i] * l[i]
                q = softmax_T(l[proposer], T)
                if cfg.mask_model >= 0:
                    M = plausibility_mask(l[cfg.mask_model], cfg.mask_alpha)
                    z = np.where(M, c / T, -np.inf)
                    m = np.max(z)
                    e = np.where(M, np.exp(z - m), 0.0)
                    r = e / np.sum(e)
                else:
                    r = softmax_T(c, T)
        else:
            # greedy: every stored logit must be a number below +inf and every model needs a
            # finite maximum, otherwise the position is reported as non-finite
            usable = bool(np.all(l < np.inf)) and bool(np.all(np.isfinite(np.max(l, axis=1))))
            q = np.zeros(V, dtype=np.float64)
            r = np.zeros(V, dtype=np.float64)
            if usable:
                q[_first_argmax(l[proposer])] = 1.0
                if cfg.combine == COMBINE_PROB_ENSEMBLE:
                    for i in range(n):
                        r[_first_argmax(l[i])] += w[i]
                else:
                    c = np.zeros(V, dtype=np.float64)
                    for i in range(n):
                        c = c + w[i] * l[i]
                    if cfg.mask_model >= 0:
                        M = plausibility_mask(l[cfg.mask_model], cfg.mask_alpha)
                        c = np.where(M, c, -np.inf)
                    usable = bool(np.isfinite(np.max(c)))
                    r[_first_argmax(c)] = 1.0
            if not usable:
                r[:] = np.nan
    ok = bool(np.all(np.isfinite(r)) and np.all(np.isfinite(q)))
    return r, q, ok


def inverse_cdf(mass: np.ndarray, u: float):
    """Index-order inverse CDF on unnormalised non-negative mass: the smallest k whose
    running sum reaches u * total; if rounding leaves u * total above every partial sum,
    the last token with positive mass.  Returns (k, total, lower_edge, upper_edge) with the
    edges normalised by total."""
    cdf = np.cumsum(mass)             # sequential, index order, float64
    total = float(cdf[-1])
    target = u * total
    k = int(np.searchsorted(cdf, target, side="left"))   # first k with cdf[k] >= target
    if k >= len(mass):
        k = int(np.nonzero(mass > 0)[0][-1])
    lo = float(cdf[k - 1]) / total if k > 0 else 0.0
    hi = float(cdf[k]) / total
    return k, total, lo, hi


# ----------------------------------------------------------------------------------------
# one (row, position)
# ----------------------------------------------------------------------------------------
@dataclass
class PositionResult:
    accept: bool = False          # meaningful for j < gamma
    cand: int = -1                # residual sample (j < gamma) or bonus sample (j == gamma)
    ratio: float = float("nan")
    r_d: float = float("nan")
    q_d: float = float("nan")
    S: float = float("nan")       # residual mass sum_x max(0, r - q)  (j < gamma)
    prob: float = float("nan")    # bonus position only: probability of cand under the law it was drawn from
    status: int = 0
    boundary_accept: bool = False
    boundary_sample: bool = False


def verify_position(l: np.ndarray, cfg: OracleConfig, proposer: int, draft: Optional[int],
                    u_acc: float, u_smp: float, return_r: bool = False, dist=None):
    """Eq. 6 at a draft position (draft is an int) or the bonus sample (draft is None).

    `dist` may carry the (r, q, ok) triple of position_distributions for these same
    arguments (with proposer = cfg.bonus_model at a bonus position that names a model), so
    that many trials on one position need not recompute it."""
    res = PositionResult()
    if draft is None and cfg.bonus_model >= 0 and dist is None:
        proposer = cfg.bonus_model               # q below is then that model's own distribution
    r, q, ok = position_distributions(l, cfg, proposer) if dist is None else dist
    if not ok:
        res.status |= STATUS_NONFINITE           # defined fallback: rejected, no candidate
        return (res, r) if return_r else res
    if draft is None:
        # Sec. 3.1: after gamma acceptances one more token is drawn; from r, or (Sec. 3.3, Algorithm 2's
        # Score) from the named model's own distribution, whose probability of it is reported
        law = q if cfg.bonus_model >= 0 else r
        k, _, lo, hi = inverse_cdf(law, u_smp)
        res.cand = k
        res.prob = float(law[k])
        res.boundary_sample = min(abs(lo - u_smp), abs(hi - u_smp)) < BOUNDARY_CDF
        return (res, r) if return_r else res
    V = l.shape[1]
    if 0 <= draft < V:
        res.r_d, res.q_d = float(r[draft]), float(q[draft])
        if res.q_d > 0.0:
            res.ratio = res.r_d / res.q_d
        else:
            res.status |= STATUS_Q_ZERO
            res.ratio = math.inf if res.r_d > 0.0 else 0.0
        thr = min(1.0, res.ratio)
        res.accept = bool(u_acc <= thr)
        res.boundary_accept = abs(u_acc - thr) < BOUNDARY_RATIO
    else:
        res.status |= STATUS_BAD_DRAFT           # never accepted; the residual is still defined
        res.accept = False
    resid = np.maximum(0.0, r - q)
    S = float(np.sum(resid))                      # reported mass; the sampler uses its own running sum
    res.S = S
    if S > 0.0:
        k, _, lo, hi = inverse_cdf(resid, u_smp)
    else:
        if not res.accept:
            res.status |= STATUS_RESIDUAL_EMPTY   # only reported when the sample is actually needed
        k, _, lo, hi = inverse_cdf(r, u_smp)
    res.cand = k
    res.boundary_sample = min(abs(lo - u_smp), abs(hi - u_smp)) < BOUNDARY_CDF
    return (res, r) if return_r else res


# ----------------------------------------------------------------------------------------
# whole batch
# ----------------------------------------------------------------------------------------
def verify(logits, dtype: str, drafts, proposer, cfg: OracleConfig, seed: int, offset: int,
           row_base: int = 0, rows: Optional[Sequence[int]] = None, return_r: bool = False,
           uniforms=None):
    """logits: array [n, B, gamma+1, V] (raw uint16 patterns when dtype == 'bf16').
    drafts [B, gamma] int; proposer [B] int, or [B, gamma+1] int naming the model that proposed each
    draft (Algorithm 2: the cached sequence holds tokens of several proposers; the entry of the bonus
    position is not read).  `rows` restricts the work to some rows
    (the others are left at their fill values), which is how full-size cases are sampled.
    `uniforms` = (u_acc, u_smp), each [B, gamma+1], replaces the Philox draws (used by the
    enumeration tests, which need to place the uniforms themselves).

    Returns a dict of arrays: accept_count [B], out_tokens [B, gamma+1] (-1 padded),
    row_status [B], bonus_prob [B] (NaN unless every draft passed), and per-position diagnostics (accept, cand, ratio, r_d, q_d, S,
    boundary_accept, boundary_sample, u_acc, u_smp), optionally r [B, gamma+1, V].
    """
    n, B, P, V = logits.shape
    g = cfg.gamma
    assert P == g + 1 and n == cfg.n and V == cfg.vocab
    drafts = np.asarray(drafts).reshape(B, g) if g > 0 else np.zeros((B, 0), np.int64)
    proposer = np.asarray(proposer)
    proposer = np.repeat(proposer.reshape(B, 1), P, axis=1) if proposer.size == B and proposer.ndim <= 1 \
        else proposer.reshape(B, P)
    if uniforms is None:
        u_acc, u_smp = position_uniforms(seed, offset, B, P, row_base)
    else:
        u_acc, u_smp = (np.asarray(x, dtype=np.float64).reshape(B, P) for x in uniforms)
    out = {
        "accept_count": np.full(B, -1, np.int32),
        "out_tokens": np.full((B, P), -1, np.int32),
        "row_status": np.zeros(B, np.uint32),
        "accept": np.zeros((B, P), bool),
        "cand": np.full((B, P), -1, np.int64),
        "ratio": np.full((B, P), np.nan), "r_d": np.full((B, P), np.nan),
        "q_d": np.full((B, P), np.nan), "S": np.full((B, P), np.nan),
        "boundary_accept": np.zeros((B, P), bool), "boundary_sample": np.zeros((B, P), bool),
        "pos_status": np.zeros((B, P), np.uint32),
        "bonus_prob": np.full(B, np.nan),
        "u_acc": u_acc, "u_smp": u_smp,
    }
    if return_r:
        out["r"] = np.full((B, P, V), np.nan)
    for b in (range(B) if rows is None else rows):
        pos = []
        for j in range(P):
            l = to_float64(logits[:, b, j, :], dtype)
            d = int(drafts[b, j]) if j < g else None
            pi = int(proposer[b, j])
            got = verify_position(l, cfg, pi, d, float(u_acc[b, j]), float(u_smp[b, j]), return_r)
            if return_r:
                got, r = got
                out["r"][b, j] = r
            pos.append(got)
            for name in ("accept", "cand", "ratio", "r_d", "q_d", "S", "boundary_accept", "boundary_sample"):
                out[name][b, j] = getattr(got, name)
            out["pos_status"][b, j] = got.status
        # first rejection (Sec. 3.1): drafts before it are kept, the position itself takes the
        # residual sample; with no rejection the bonus sample of position gamma is appended.
        a = g
        for j in range(g):
            if not pos[j].accept:
                a = j
                break
        out["accept_count"][b] = a
        out["out_tokens"][b, :a] = drafts[b, :a]
        out["out_tokens"][b, a] = pos[a].cand
        if a == g:
            out["bonus_prob"][b] = pos[g].prob
        st = 0
        for j in range(a + 1):                    # positions after the first rejection are discarded
            st |= pos[j].status
        out["row_status"][b] = st
    return out


# ----------------------------------------------------------------------------------------
# closed forms used by the tests and reports (Eq. 7; App. A.1)
# ----------------------------------------------------------------------------------------
def acceptance_rate(r: np.ndarray, q: np.ndarray) -> float:
    """alpha = 1 - 1/2 * sum_x |q(x) - r(x)|  (Eq. 7, with the paper's D_TV = sum |q - r|)."""
    return 1.0 - 0.5 * float(np.sum(np.abs(q - r)))
