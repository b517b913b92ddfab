"""A tiny deterministic language model and an n-gram draft table, in float64 numpy.

TEST INFRASTRUCTURE ONLY (part of the CPU oracle).  The model exists so that the claim
"greedy speculative decoding emits exactly the tokens of one-token-at-a-time greedy
decoding" (Sec. 2.3, speculative decoding) can be checked end to end: one attention layer
whose attention is supplied by a backend (the oracle's, or the CUDA library's in GPU tests),
with seeded projections around it.

The n-gram table follows Sec. 4.3: slide a window of n tokens over a token stream, key = the
first n-1 tokens, value = the successor seen most often with that key.  The paper does not
say which successor wins a count tie; here the lowest token id wins (a rule that does not
depend on the order in which windows are visited).
"""
from __future__ import annotations

from collections import OrderedDict

import numpy as np


class ToyLM:
    """x = E[token] + Ppos[pos];  q,k,v = x Wq, x Wk, x Wv (rounded to float32 storage);
    h = x + concat_heads(attn) Wo;  logits = h E^T.  All weights seeded N(0,1)/sqrt(fan_in)."""

    def __init__(self, seed: int = 11, vocab: int = 512, width: int = 64, num_q_heads: int = 4,
                 num_kv_heads: int = 2, head_dim: int = 64, max_pos: int = 1024, gain: float = 4.0):
        rng = np.random.default_rng(seed)
        self.vocab, self.width = vocab, width
        self.hq, self.hkv, self.d = num_q_heads, num_kv_heads, head_dim
        self.E = rng.standard_normal((vocab, width))
        self.Ppos = rng.standard_normal((max_pos, width)) * 0.5
        s = 1.0 / np.sqrt(width)
        self.Wq = rng.standard_normal((width, num_q_heads * head_dim)) * s * gain
        self.Wk = rng.standard_normal((width, num_kv_heads * head_dim)) * s
        self.Wv = rng.standard_normal((width, num_kv_heads * head_dim)) * s
        self.Wo = rng.standard_normal((num_q_heads * head_dim, width)) / np.sqrt(num_q_heads * head_dim) * gain

    def embed(self, tokens, positions) -> np.ndarray:
        return self.E[np.asarray(tokens)] + self.Ppos[np.asarray(positions)]

    def qkv(self, x: np.ndarray):
        """Returns float32 storage arrays q [n,Hq,d], k [n,Hkv,d], v [n,Hkv,d]."""
        n = x.shape[0]
        q = (x @ self.Wq).reshape(n, self.hq, self.d).astype(np.float32)
        k = (x @ self.Wk).reshape(n, self.hkv, self.d).astype(np.float32)
        v = (x @ self.Wv).reshape(n, self.hkv, self.d).astype(np.float32)
        return q, k, v

    def logits(self, x: np.ndarray, attn_out: np.ndarray) -> np.ndarray:
        """attn_out [n,Hq,d] float64 -> float32 storage logits [n, vocab]."""
        n = x.shape[0]
        h = x + attn_out.reshape(n, -1).astype(np.float64) @ self.Wo
        return (h @ self.E.T).astype(np.float32)


def build_ngram_table(stream, n: int = 3) -> dict:
    """Sec. 4.3: slide a window of n tokens over the stream; key = its first n-1 tokens, value = the
    successor recorded most often with that key.  Equal counts: the lowest token id wins."""
    stream = [int(t) for t in stream]
    counts: dict = {}
    for i in range(len(stream) - n + 1):
        key = tuple(stream[i:i + n - 1])
        nxt = stream[i + n - 1]
        bucket = counts.setdefault(key, {})
        bucket[nxt] = bucket.get(nxt, 0) + 1
    table = {}
    for key, bucket in counts.items():
        top = max(bucket.values())
        table[key] = min(tok for tok, c in bucket.items() if c == top)
    return table


def ngram_drafts(table: dict, history, k: int, n: int, rng=None, vocab: int = 0, fill=None):
    """Sec. 4.3: chain k drafts from the last n-1 tokens.  Returns None when the FIRST lookup
    misses (selective fallback to a plain one-token step); a later miss guesses a token: ``fill[i]``
    when given, else a draw from ``rng``."""
    ctx = [int(t) for t in history[-(n - 1):]]
    if len(ctx) < n - 1 or tuple(ctx) not in table:
        return None
    out = []
    for i in range(k):
        tok = table.get(tuple(ctx))
        if tok is None:
            tok = int(fill[i]) if fill is not None else int(rng.integers(0, vocab))
        out.append(int(tok))
        ctx = (ctx + [int(tok)])[1:] if n > 1 else []
    return out
