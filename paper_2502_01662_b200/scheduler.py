"""The schedulers of the paper around the verification step: the alternate proposal framework for two
models (Sec. 3.3, Algorithm 1) and its n-model form (App. B, Algorithm 2).

Two models take turns.  In a cycle the proposer extends the cached token (if any) to its proposal
length, the verifier scores the proposal, and one verification call decides: the accepted prefix is
kept; at the first rejection the position is resampled from the residual and the cache is cleared;
when every draft passes, the verifier's bonus token -- drawn from the verifier's own distribution,
not from the combined one -- is cached and becomes the first token of the verifier's own proposal in
the next cycle, where the roles are swapped.  A token therefore reaches the output only through the
accept test against the combined distribution, which is why the output follows that distribution.

The verification call is passed in (`verify`): the product path hands in `gpu_verify(...)`, which runs
the CUDA library; this module holds no verification arithmetic of its own.  The models are stand-ins:
`TableModel` maps a context (last token, position) to a row of a seeded logit table, so that every
call is reproducible on any machine.
"""
from __future__ import annotations

from dataclasses import dataclass, field
from typing import Callable, List, Optional, Sequence, Tuple

import numpy as np

# verify(logits[n, 1, g+1, V] float32, drafts[1, g] int32, proposer, bonus_model, seed, offset)
#   -> (accept_count, out_tokens[g+1], bonus_prob)
# proposer: one model index for the row, or an int32 table [1, g+1] naming the proposer of every draft;
# bonus_model: -1 (bonus from the combined distribution) or the model whose own distribution it follows
VerifyFn = Callable[[np.ndarray, np.ndarray, object, int, int, int], Tuple[int, np.ndarray, float]]


class TableModel:
    """A stand-in for a language model: next-token logits looked up in a seeded table.

    `contexts` rows; the row is chosen from the last token and the position, so the logits change
    along a sequence but any prefix gives the same answer everywhere.  contexts = 1 makes the model
    ignore its input, which gives every position the same acceptance rate (the setting of the
    closed forms of Sec. 3.2 and 3.3)."""

    def __init__(self, table: np.ndarray):
        self.table = np.ascontiguousarray(table, dtype=np.float32)   # [contexts, V]
        self.contexts, self.vocab = self.table.shape
        self.calls = 0            # forward passes (one per scored sequence or proposed token)

    def context_of(self, prefix: Sequence[int]) -> int:
        last = prefix[-1] if len(prefix) else 0
        return (int(last) * 2654435761 + len(prefix) * 40503) % self.contexts

    def logits(self, prefix: Sequence[int]) -> np.ndarray:
        return self.table[self.context_of(prefix)]


def make_table_models(n: int, vocab: int, contexts: int, seed: int, sigma: float = 2.0, rho: float = 0.8) -> List[TableModel]:
    """n correlated table models: l_i = sigma * (sqrt(rho) z + sqrt(1 - rho) e_i), z shared."""
    g = np.random.Generator(np.random.Philox(key=seed))
    z = g.standard_normal((contexts, vocab))
    return [TableModel(sigma * (np.sqrt(rho) * z + np.sqrt(1.0 - rho) * g.standard_normal((contexts, vocab))))
            for _ in range(n)]


@dataclass
class CycleRecord:
    proposer: int
    cached: int            # tokens taken over from the previous cycle's bonus (0 or 1)
    drafts: List[int]
    accept_count: int
    emitted: List[int]
    bonus: Optional[int]   # cached for the next cycle, when every draft passed


@dataclass
class Stats:
    cycles: int = 0
    tokens: int = 0
    proposed: int = 0              # proposer forward passes (tokens it generated itself)
    scored: int = 0                # verifier forward passes (one per cycle)
    full_accepts: int = 0
    history: List[CycleRecord] = field(default_factory=list)


class AlternateProposal:
    """Algorithm 1.  models = (M_q, M_p): M_q is the default proposer; gammas = (gamma_q, gamma_p)."""

    def __init__(self, models: Sequence[TableModel], gammas: Sequence[int], temperature: float, verify: VerifyFn,
                 propose_seed: int = 1, verify_seed: int = 2, keep_history: bool = False):
        if len(models) != 2 or len(gammas) != 2 or min(gammas) < 1:
            raise ValueError("two models and two proposal lengths >= 1")
        if models[0].vocab != models[1].vocab:
            raise ValueError("the models must share a vocabulary")
        self.models, self.gammas, self.T = list(models), list(gammas), float(temperature)
        self.verify = verify
        self.verify_seed = verify_seed
        self._u = np.random.Generator(np.random.Philox(key=propose_seed))
        self.keep_history = keep_history

    # Propose: one token from model i after `prefix`, at the temperature of the run
    def _propose_one(self, i: int, prefix: Sequence[int]) -> int:
        m = self.models[i]
        m.calls += 1
        l = m.logits(prefix).astype(np.float64)
        if self.T == 0.0:
            return int(np.argmax(l))
        z = l / self.T
        p = np.exp(z - z.max())
        cdf = np.cumsum(p)
        k = int(np.searchsorted(cdf, self._u.random() * cdf[-1], side="left"))
        return min(k, m.vocab - 1)

    def generate(self, prefix: Sequence[int], max_new_tokens: int) -> Tuple[List[int], Stats]:
        S: List[int] = list(prefix)
        C: List[int] = []                       # cached bonus token of the previous cycle
        proposer, verifier = 0, 1
        st = Stats()
        V = self.models[0].vocab
        while st.tokens < max_new_tokens:
            if not C:
                proposer, verifier = 0, 1       # standard speculative step: the default proposer
            else:
                proposer, verifier = verifier, proposer
            g = self.gammas[proposer]
            T = list(C)
            while len(T) < g:                   # the proposer completes its proposal
                T.append(self._propose_one(proposer, S + T))
                st.proposed += 1
            # Score: both models' logits at the gamma draft positions and after the last draft (the
            # proposer's are known from proposing; the verifier's come from one pass over S + T)
            self.models[verifier].calls += 1
            st.scored += 1
            logits = np.empty((2, 1, g + 1, V), dtype=np.float32)
            for j in range(g + 1):
                ctx = S + T[:j]
                logits[0, 0, j] = self.models[0].logits(ctx)
                logits[1, 0, j] = self.models[1].logits(ctx)
            drafts = np.asarray(T, dtype=np.int32).reshape(1, g)
            a, out, prob = self.verify(logits, drafts, proposer, verifier, self.verify_seed, st.cycles)
            emitted = [int(x) for x in out[: a + 1]] if a < g else [int(x) for x in out[:g]]
            bonus = int(out[g]) if a == g else None
            if self.keep_history:
                st.history.append(CycleRecord(proposer, len(C), list(T), int(a), emitted, bonus))
            S += emitted
            st.tokens += len(emitted)
            st.cycles += 1
            if a == g:
                st.full_accepts += 1
                C = [bonus]                     # the verifier's own token: its next proposal starts with it
            else:
                C = []                          # a rejection invalidates everything cached
        return S[len(prefix):], st


@dataclass
class Event:
    kind: str              # "propose", "score", "verify"
    model: int             # the model that proposed / scored; -1 for verify
    count: int             # tokens proposed, cached tokens scored, or tokens verified
    accepted: int = -1     # verify only


class CollaborativeSpeculation:
    """Algorithm 2: n models, proposal lengths gamma_1..gamma_n, model 0 the default proposer.

    S_c is the cached sequence, `owner[k]` the model that produced its k-th token, `scored[i]` how many
    of its tokens model i has probabilities for (its own proposals count).  The model with the fewest
    scores the whole cache, which also yields its bonus token (drawn from its own distribution, with its
    probability); every cached token that all models have scored is then verified against the combined
    distribution, its proposer's distribution being q -- one verification call for the whole verifiable
    prefix, which stops at the first rejection exactly as the token-by-token loop of the listing does.
    After a rejection everything cached is dropped and the default proposer starts over (the reading of
    Sec. 3.3 and of the walk-through in App. B; the listing would let the scoring model propose first)."""

    def __init__(self, models: Sequence[TableModel], gammas: Sequence[int], temperature: float, verify: VerifyFn,
                 propose_seed: int = 1, verify_seed: int = 2, keep_events: bool = False):
        if len(models) < 2 or len(models) != len(gammas) or min(gammas) < 1:
            raise ValueError("n >= 2 models and one proposal length >= 1 for each")
        self.models, self.gammas, self.T = list(models), list(gammas), float(temperature)
        self.n, self.V = len(models), models[0].vocab
        self.verify, self.verify_seed = verify, verify_seed
        self._u = np.random.Generator(np.random.Philox(key=propose_seed))
        self.keep_events = keep_events
        self.events: List[Event] = []
        self.calls = 0         # verification calls so far: the counter offset of the next one

    def _log(self, *a):
        if self.keep_events:
            self.events.append(Event(*a))

    def _sample(self, i: int, prefix: Sequence[int]) -> int:
        m = self.models[i]
        m.calls += 1
        l = m.logits(prefix).astype(np.float64)
        if self.T == 0.0:
            return int(np.argmax(l))
        z = l / self.T
        p = np.exp(z - z.max())
        cdf = np.cumsum(p)
        return min(int(np.searchsorted(cdf, self._u.random() * cdf[-1], side="left")), self.V - 1)

    def generate(self, prefix: Sequence[int], max_new_tokens: int) -> Tuple[List[int], Stats]:
        n, V = self.n, self.V
        S: List[int] = list(prefix)
        Sc: List[int] = []
        owner: List[int] = []
        scored = [0] * n
        st = Stats()
        start = len(prefix)

        def propose(i: int, count: int):
            for _ in range(count):
                Sc.append(self._sample(i, S + Sc))
                owner.append(i)
                st.proposed += 1
            scored[i] = len(Sc)      # a model knows its own probabilities along everything it has seen
            self._log("propose", i, count)

        while len(S) - start < max_new_tokens:
            if not Sc:
                propose(0, self.gammas[0])
                continue
            i = int(np.argmin(scored))                    # fewest cached probabilities; lowest index on ties
            # Score: model i reads the whole cache (one forward pass) and draws its bonus token from its own
            # distribution after it; the probability comes back with the token
            self.models[i].calls += 1
            st.scored += 1
            self._log("score", i, len(Sc))
            row = self.models[i].logits(S + Sc)
            lg = np.broadcast_to(row, (n, 1, 1, V)).astype(np.float32).copy()
            _, out, prob = self.verify(lg, np.zeros((1, 0), np.int32), 0, i, self.verify_seed, self.calls)
            self.calls += 1
            Sc.append(int(out[0]))
            owner.append(i)
            scored[i] = len(Sc)
            # Verify every cached token that all models have scored
            L = min(scored)
            rejected = False
            if L > 0:
                lg = np.empty((n, 1, L + 1, V), dtype=np.float32)
                for j in range(L + 1):                    # position L only fills the call's bonus slot, unused here
                    ctx = S + Sc[:j]
                    for k in range(n):
                        lg[k, 0, j] = self.models[k].logits(ctx)
                table = np.asarray(owner[:L] + [0], dtype=np.int32).reshape(1, L + 1)
                a, out, _ = self.verify(lg, np.asarray(Sc[:L], np.int32).reshape(1, L), table, -1, self.verify_seed,
                                        self.calls)
                self.calls += 1
                self._log("verify", -1, L, int(a))
                st.cycles += 1
                if a == L:
                    S += Sc[:L]
                    del Sc[:L], owner[:L]
                    scored = [c - L for c in scored]
                    st.full_accepts += 1
                else:
                    S += Sc[:a] + [int(out[a])]           # the resampled token replaces the rejected one
                    Sc.clear()
                    owner.clear()
                    scored = [0] * n
                    rejected = True
            if not rejected:
                propose(i, self.gammas[i] - 1)            # the bonus token was the first of model i's proposal
        st.tokens = len(S) - start
        return S[start:], st


def gpu_verify(combine: int, weights: Sequence[float], temperature: float, vocab: int, mask_model: int = -1,
               mask_alpha: float = 1.0, device: int = 0) -> VerifyFn:
    """The verification call of the CUDA library for the schedulers: one context per proposal length,
    made on first use, host tensors in and out (cos_verify_run_host)."""
    import torch
    from .binding import CosVerifier
    ctxs = {}
    n = len(list(weights))

    def verify(logits, drafts, proposer, bonus_model, seed, offset):
        g = logits.shape[2] - 1
        if g not in ctxs:
            ctxs[g] = CosVerifier(n, combine, weights, temperature, g, vocab, 1, torch.float32, mask_model=mask_model,
                                  mask_alpha=mask_alpha, device=device, host_staging=True)
        prop = torch.tensor([proposer], dtype=torch.int32) if np.isscalar(proposer) else \
            torch.from_numpy(np.ascontiguousarray(proposer, dtype=np.int32))
        outs = ctxs[g].run_host(torch.from_numpy(logits), torch.from_numpy(drafts) if g > 0 else None,
                                prop, seed, offset, bonus_model=bonus_model)
        return int(outs["accept_count"][0]), outs["out_tokens"][0].numpy().copy(), float(outs["bonus_prob"][0])

    verify.close = lambda: [c.close() for c in ctxs.values()]
    return verify
