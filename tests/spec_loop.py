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


class CudaBackend:
    """The same cache and step on the GPU: agx_kv_append, agx_attn_prefixed and agx_accept_greedy through the
    C ABI (float32 pools); the toy model's projections around them stay in numpy."""

    def __init__(self, lm, max_tokens=512, seed=5):
        import torch
        from paper_2605_10380_b200 import agx
        self.torch, self.lm = torch, lm
        self.h = agx.Handle(lm.hq, lm.hkv, lm.d, "f32")
        n_pages = (max_tokens + 15) // 16
        rng = np.random.default_rng(seed)
        self.page_row = rng.permutation(n_pages + 8).astype(np.int32)[:n_pages]
        self.page_table = torch.from_numpy(self.page_row[None, :].copy()).cuda()
        self.k_pool = torch.zeros((n_pages + 8, lm.hkv, 16, lm.d), dtype=torch.float32, device="cuda")
        self.v_pool = torch.zeros_like(self.k_pool)
        self.length = 0

    def run_block(self, tokens, drafts):
        torch = self.torch
        n, P = len(tokens), self.length
        x = self.lm.embed(tokens, np.arange(P, P + n))
        q, k, v = self.lm.qkv(x)
        dq, dk, dv = (torch.from_numpy(a).cuda() for a in (q, k, v))
        cu = torch.tensor([0, n], dtype=torch.int32, device="cuda")
        pl = torch.tensor([P], dtype=torch.int32, device="cuda")
        self.h.kv_append(self.k_pool, self.v_pool, dk, dv, self.page_table, pl, cu)
        out = torch.empty_like(dq)
        Pn, Qn = np.array([P], np.int32), np.array([n], np.int32)
        nws = self.h.attn_workspace_bytes(Pn, Qn)
        ws = torch.empty(max(nws, 256), dtype=torch.uint8, device="cuda") if nws else None
        self.h.attn_prefixed(dq, self.k_pool, self.v_pool, self.page_table, Pn, Qn, out, None, ws)
        logits = torch.from_numpy(self.lm.logits(x, out.cpu().numpy().astype(np.float64))).cuda()
        dd = torch.tensor(list(drafts) if len(drafts) else [0], dtype=torch.int32, device="cuda")
        acc = torch.zeros(1, dtype=torch.int32, device="cuda"); nxt = torch.zeros(1, dtype=torch.int32, device="cuda")
        sl = pl.clone()
        aws = torch.empty(self.h.accept_workspace_bytes(n, self.lm.vocab), dtype=torch.uint8, device="cuda")
        self.h.accept_greedy(logits, "f32", self.lm.vocab, dd, cu, acc, nxt, None, sl, aws)
        torch.cuda.synchronize()
        self.length = int(sl.item())
        return int(acc.item()), int(nxt.item())


class DeviceNgramDrafts:
    """Draft source on the GPU: agx_ngram_build once over the prompt, agx_ngram_draft per round
    (Sec. 4.3, with the selective fallback)."""

    def __init__(self, prompt, n=3, seed=3, vocab=512):
        import torch
        from paper_2605_10380_b200 import agx
        self.torch, self.n, self.vocab = torch, n, vocab
        self.h = agx.Handle(4, 2, 64, "f32")
        st = torch.tensor([int(t) for t in prompt], dtype=torch.int32, device="cuda")
        self.lut = torch.empty(agx.ngram_lut_bytes(len(prompt)), dtype=torch.uint8, device="cuda")
        ws = torch.empty(agx.ngram_workspace_bytes(len(prompt)), dtype=torch.uint8, device="cuda")
        self.h.ngram_build(st, n, self.lut, ws)
        self.rng = np.random.default_rng(seed)

    def __call__(self, history, k):
        torch = self.torch
        ctx = torch.tensor([int(t) for t in history[-(self.n - 1):]], dtype=torch.int32, device="cuda").reshape(1, self.n - 1)
        fill = torch.from_numpy(self.rng.integers(0, self.vocab, size=(1, k)).astype(np.int32)).cuda()
        drafts = torch.zeros((1, k), dtype=torch.int32, device="cuda")
        has = torch.zeros(1, dtype=torch.int32, device="cuda")
        self.h.ngram_draft(self.lut, ctx, fill, k, drafts, has)
        return drafts[0].tolist() if has.item() else None


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
