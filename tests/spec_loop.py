"""Harness: a greedy generation loop over a toy LM, one token at a time or with draft groups.

The loop is control flow only (Sec. 2.3 speculative decoding rounds; Sec. 4.3 selective
fallback).  Attention, KV append and acceptance come from a backend object so the same loop
drives the CPU oracle and the CUDA library.
"""
from __future__ import annotations

import numpy as np


class OracleBackend:
    """KV cache of one sequence in a paged float32 pool, served by the CPU oracle."""

    def __init__(self, lm, max_tokens=512, seed=5):
        import oracle
        self.o = oracle
        self.lm = lm
        n_pages = (max_tokens + 15) // 16
        rng = np.random.default_rng(seed)
        self.page_row = rng.permutation(n_pages + 8).astype(np.int32)[:n_pages]
        self.k_pool = np.zeros((n_pages + 8, lm.hkv, 16, lm.d), dtype=np.float32)
        self.v_pool = np.zeros_like(self.k_pool)
        self.length = 0

    def step(self, q, k, v, drafts):
        """Append the block at the committed length, attend, compute logits, accept.
        Returns (accept_len, next_token)."""
        n = q.shape[0]
        P = self.length
        cu = np.array([0, n], dtype=np.int32)
        pl = np.array([P], dtype=np.int32)
        self.o.kv_append(self.k_pool, self.v_pool, k, v, "f32", self.page_row[None, :], pl, cu)
        out, _, _ = self.o.attn_paged(q, self.k_pool, self.v_pool, self.page_row, "f32", P)
        logits = self.lm.logits(self._x, out)
        am, al, nt, sl = self.o.accept_greedy(logits, "f32", self.lm.vocab,
                                              np.asarray(drafts, dtype=np.int32), cu, pl)
        self.length = int(sl[0])
        return int(al[0]), int(nt[0])

    def run_block(self, tokens, drafts):
        pos = np.arange(self.length, self.length + len(tokens))
        self._x = self.lm.embed(tokens, pos)
        q, k, v = self.lm.qkv(self._x)
        return self.step(q, k, v, drafts)


def generate(backend, prompt, n_new, draft_fn=None, k=4):
    """Greedy generation.  ``draft_fn(history, k)`` returns k draft tokens or None (plain step).
    Returns (emitted tokens, number of model calls, list of accept lengths)."""
    prompt = [int(t) for t in prompt]
    # prefill: the whole prompt is one block with zero drafts taken from its last row only
    # (rows before the last are prompt positions, not drafts), so feed prompt[:-1] then the tail.
    if len(prompt) > 1:
        backend.run_block(prompt[:-1], [0] * (len(prompt) - 2))
        backend.length = len(prompt) - 1  # prompt tokens are given, not speculative
    history = list(prompt)
    emitted, calls, accepts = [], 0, []
    while len(emitted) < n_new:
        drafts = draft_fn(history, k) if draft_fn is not None else None
        if drafts is None:
            a, nxt = backend.run_block([history[-1]], [])
            new = [nxt]
        else:
            a, nxt = backend.run_block([history[-1]] + list(drafts), list(drafts))
            new = list(drafts[:a]) + [nxt]
            accepts.append(a)
        calls += 1
        emitted.extend(new)
        history.extend(new)
    return emitted[:n_new], calls, accepts
