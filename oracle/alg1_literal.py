"""Algorithm 1 kept in the paper's own data structures (numpy, fp64) — TEST INFRASTRUCTURE ONLY.

The attention message is a bool matrix with one row per recent query and one column per cached key, exactly as the
paper's eviction routine holds it; the C oracle re-encodes the same information as a shift register per key and the
tests require both to agree. Two repairs to the printed routine are taken: the new verdict is appended as a row
(the printed concatenation axis cannot work for shapes [m, l] and [1, l]), and the message columns are gathered
together with the keys and values so that the next call's [m, l-1] contract holds.
"""
from __future__ import annotations

import numpy as np


class LiteralUnit:
    """One KV head with its group of G query heads, state held as (keys, values, message, pos)."""

    def __init__(self, head_dim, w, r, alpha):
        self.d, self.w, self.r, self.alpha = head_dim, w, r, float(alpha)
        self.keys = np.zeros((0, head_dim))
        self.values = np.zeros((0, head_dim))
        self.message = np.zeros((0, 0), dtype=bool)
        self.pos = np.zeros((0,), dtype=np.int64)
        self.t = 0

    def _attention_row(self, qv, n):
        """Eq. 2 over the first n cached keys."""
        logits = self.keys[:n] @ qv / np.sqrt(self.d)
        e = np.exp(logits - logits.max())
        return e / e.sum()

    def _record_and_evict(self, verdict_row):
        """Algorithm 1: append the verdict row, keep the last w rows, evict once w rows exist."""
        l = self.keys.shape[0]
        m = self.message.shape[0]
        message = np.concatenate([self.message, np.zeros((m, l - self.message.shape[1]), dtype=bool)], axis=1)
        message = np.concatenate([message, verdict_row[None, :]], axis=0)[-self.w:, :]
        if message.shape[0] >= self.w:
            decision = message.any(axis=0)
            decision[-self.r:] = True                      # the r most recent tokens always stay
            idx = np.nonzero(decision)[0]
            self.keys, self.values, self.pos = self.keys[idx], self.values[idx], self.pos[idx]
            message = message[:, idx]
        self.message = message

    def decode_step(self, q_group, k_new, v_new):
        """q_group [G, d]; returns out [G, d] computed on the cache before this step's eviction."""
        self.t += 1
        self.keys = np.concatenate([self.keys, np.asarray(k_new, dtype=np.float64)[None]], axis=0)
        self.values = np.concatenate([self.values, np.asarray(v_new, dtype=np.float64)[None]], axis=0)
        self.pos = np.concatenate([self.pos, [self.t]])
        l = self.keys.shape[0]
        verdict = np.zeros((l,), dtype=bool)
        outs = []
        for qv in np.asarray(q_group, dtype=np.float64):
            attn = self._attention_row(qv, l)
            outs.append(attn @ self.values)
            verdict |= attn >= self.alpha / self.t           # Definition 3.1; OR over the group (GQA rule)
        self._record_and_evict(verdict)
        return np.stack(outs)

    def compress_prompt(self, k_prompt, v_prompt, q_last_group):
        """k_prompt/v_prompt [P, d]; q_last_group [G, w, d] = queries of positions P-w+1..P (rows before position 1
        are ignored). Rows are recorded oldest first through the same routine as a decode step; since eviction needs
        w rows, only the last row can evict, so every row sees the full prompt."""
        P = k_prompt.shape[0]
        self.keys = np.asarray(k_prompt, dtype=np.float64).copy()
        self.values = np.asarray(v_prompt, dtype=np.float64).copy()
        self.pos = np.arange(1, P + 1)
        self.message = np.zeros((0, P), dtype=bool)
        self.t = P
        wp = min(P, self.w)
        for row in range(self.w - wp, self.w):
            i = P - (self.w - 1 - row)
            verdict = np.zeros((self.keys.shape[0],), dtype=bool)
            for qg in np.asarray(q_last_group, dtype=np.float64):
                attn = self._attention_row(qg[row], i)          # causal row: keys 1..i of the untouched prompt
                verdict[:i] |= attn >= self.alpha / i           # keys newer than the query keep a 0 bit
            self._record_and_evict(verdict)                     # evicts only once w rows exist: at the last row

    def ages(self):
        """Per cached key: how many recorded queries ago it was last found important (0 = latest), -1 if never."""
        m, l = self.message.shape
        out = np.full((l,), -1, dtype=np.int32)
        for b in range(m - 1, -1, -1):                    # oldest candidate first, newest overwrites
            out[self.message[m - 1 - b]] = b
        return out

    def words(self):
        """Shift-register view of the message: bit b = verdict of the query b steps ago."""
        m, l = self.message.shape
        out = np.zeros((l,), dtype=np.uint32)
        for b in range(m):
            out |= self.message[m - 1 - b].astype(np.uint32) << np.uint32(b)
        return out
