"""A second, independent statement of the recent-message policy (numpy, fp64) — TEST INFRASTRUCTURE ONLY.

Every cached key is a record that remembers WHICH queries judged it important: the set of query indices (queries are
numbered as they are recorded, prompt rows included). Nothing here is a matrix or a shift register. The policy reads
off the definitions: a key is long-term minor when none of the last w recorded queries is in its set (Definition 4.1
with the window of the "Approach" paragraph); once w queries have been recorded, long-term minor keys are dropped,
except the r newest entries of the cache (Algorithm 1's protected tail). The C oracle keeps a w-bit shift register
per key instead; the tests require both to agree on live lists, rows, and on what the registers can still say.
"""
from __future__ import annotations

import numpy as np


class _Entry:
    __slots__ = ("pos", "k", "v", "liked_by")

    def __init__(self, pos, k, v):
        self.pos, self.k, self.v = pos, np.asarray(k, dtype=np.float64), np.asarray(v, dtype=np.float64)
        self.liked_by = set()                      # indices of the recorded queries that found this key important


class HistoryUnit:
    """One KV head with its group of G query heads."""

    def __init__(self, head_dim, w, r, alpha):
        self.d, self.w, self.r, self.alpha = head_dim, w, r, float(alpha)
        self.entries = []                          # oldest first
        self.t = 0                                 # tokens seen
        self.n_queries = 0                         # queries recorded so far (index of the latest one)

    # ---- views the tests compare ----
    @property
    def pos(self):
        return np.array([e.pos for e in self.entries], dtype=np.int64)

    @property
    def keys(self):
        return np.array([e.k for e in self.entries], dtype=np.float64).reshape(len(self.entries), self.d)

    @property
    def values(self):
        return np.array([e.v for e in self.entries], dtype=np.float64).reshape(len(self.entries), self.d)

    def _recent_queries(self):
        """Indices of the last w recorded queries."""
        return range(max(1, self.n_queries - self.w + 1), self.n_queries + 1)

    def ages(self):
        """Per cached key: how many recorded queries ago it was last found important (0 = latest), -1 if by none of
        the last w."""
        window = set(self._recent_queries())
        out = []
        for e in self.entries:
            seen = e.liked_by & window
            out.append(self.n_queries - max(seen) if seen else -1)
        return np.array(out, dtype=np.int32)

    def words(self):
        """What a w-bit (w <= 32) shift register would hold: bit b = verdict of the query b steps ago."""
        out = []
        for e in self.entries:
            out.append(sum(1 << (self.n_queries - i) for i in self._recent_queries() if i in e.liked_by))
        return np.array(out, dtype=np.uint32)

    # ---- the method ----
    def _probabilities(self, qv, entries):
        """Eq. 2 of one query over the given entries."""
        logits = np.array([e.k @ qv for e in entries]) / np.sqrt(self.d)
        e = np.exp(logits - logits.max())
        return e / e.sum()

    def _record(self, liked):
        """One more query is on record; `liked` are the entries it found important. Then the policy."""
        self.n_queries += 1
        for e in liked:
            e.liked_by.add(self.n_queries)
        if self.n_queries < self.w:                # fewer than w queries on record: nothing is judged long-term minor yet
            return
        window = set(self._recent_queries())
        protected = set(id(e) for e in self.entries[-self.r:])
        self.entries = [e for e in self.entries if (e.liked_by & window) or id(e) in protected]

    def decode_step(self, q_group, k_new, v_new):
        """q_group [G, d]; returns out [G, d] computed on the cache before this step's eviction."""
        self.t += 1
        self.entries.append(_Entry(self.t, k_new, v_new))
        liked, outs = [], []
        vals = self.values
        for qv in np.asarray(q_group, dtype=np.float64):
            p = self._probabilities(qv, self.entries)
            outs.append(p @ vals)                                              # Eq. 1
            liked += [e for e, pj in zip(self.entries, p) if pj >= self.alpha / self.t]   # Definition 3.1, any head of the group
        self._record(liked)
        return np.stack(outs)

    def compress_prompt(self, k_prompt, v_prompt, q_last_group):
        """k_prompt/v_prompt [P, d]; q_last_group [G, w, d] = queries of positions P-w+1..P (rows that would fall
        before position 1 are ignored). The query at position i sees keys 1..i of the untouched prompt with the
        threshold alpha/i; the policy runs after each recorded query, so it can only fire at the last one."""
        P = k_prompt.shape[0]
        self.entries = [_Entry(j + 1, k_prompt[j], v_prompt[j]) for j in range(P)]
        self.t, self.n_queries = P, 0
        q_last_group = np.asarray(q_last_group, dtype=np.float64)
        for i in range(max(1, P - self.w + 1), P + 1):
            row = self.w - 1 - (P - i)
            causal = self.entries[:i]                                         # nothing has been dropped yet
            liked = []
            for qg in q_last_group:
                p = self._probabilities(qg[row], causal)
                liked += [e for e, pj in zip(causal, p) if pj >= self.alpha / i]
            self._record(liked)
