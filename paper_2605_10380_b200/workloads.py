"""Seeded synthetic inputs for the prefix-cached block-attention / greedy-accept path.

This module only draws random numbers, rounds them to a storage dtype and lays them out
(page pools, page tables, ragged offsets, draft plans).  It holds none of the method's
arithmetic: no dot product, no softmax, no argmax.  Both the CUDA path's tests/benchmarks
and the CPU oracle's tests take their inputs from here, so the two sides see bit-identical
data without sharing any code that computes a result.

Storage conventions
-------------------
* ``dtype == "bf16"``: arrays are ``uint16`` holding bfloat16 bit patterns.
* ``dtype == "f32"`` : arrays are ``float32``.
* KV pools are ``[num_pages, Hkv, PAGE, d]`` (PAGE = 16); logical token ``t`` of sequence
  ``s`` lives in page ``page_table[s, t // 16]`` at slot ``t % 16``.
* Ragged batches use ``cu_q`` (``[B+1]`` exclusive prefix sum of ``q_len``); rows of
  ``q_block`` / ``k_new`` / ``v_new`` / ``logits`` are sequence-major, position-minor.
* ``drafts`` is ``[total_q - B]``: sequence ``s`` owns ``q_len[s] - 1`` consecutive entries
  starting at ``cu_q[s] - s``.

The five named configurations mirror the shapes of on-device agent workloads (a 7B-class
GQA 32/8, head_dim 128 model; a ~3k-token cached system-prompt/tool prefix with a ~512-token
uncached suffix; short draft groups), with i.i.d. N(0,1) values standing in for real
activations.
"""
from __future__ import annotations

from dataclasses import dataclass, field
from typing import Optional

import numpy as np

PAGE = 16


# --------------------------------------------------------------------------- dtype helpers
def f32_to_bf16_bits(x: np.ndarray) -> np.ndarray:
    """Round float32 to bfloat16 (round-to-nearest-even) and return the uint16 bit patterns."""
    x = np.ascontiguousarray(x, dtype=np.float32)
    u = x.view(np.uint32)
    nan = np.isnan(x)
    rounded = (u + (np.uint32(0x7FFF) + ((u >> np.uint32(16)) & np.uint32(1)))) >> np.uint32(16)
    out = rounded.astype(np.uint16)
    if nan.any():
        out[nan] = np.uint16(0x7FC0)
    return out


def bf16_bits_to_f32(b: np.ndarray) -> np.ndarray:
    """Widen bfloat16 bit patterns (uint16) to float32 exactly."""
    b = np.ascontiguousarray(b, dtype=np.uint16)
    return (b.astype(np.uint32) << np.uint32(16)).view(np.float32)


def to_storage(x_f32: np.ndarray, dtype: str) -> np.ndarray:
    if dtype == "bf16":
        return f32_to_bf16_bits(x_f32)
    if dtype == "f32":
        return np.ascontiguousarray(x_f32, dtype=np.float32)
    raise ValueError(f"unknown dtype {dtype!r}")


def storage_to_f32(x: np.ndarray, dtype: str) -> np.ndarray:
    """Exact widening of a storage array to float32 (bf16 and f32 both embed in f32)."""
    if dtype == "bf16":
        return bf16_bits_to_f32(x)
    return np.ascontiguousarray(x, dtype=np.float32)


def _normal_storage(rng: np.random.Generator, shape, dtype: str, chunk_rows: int = 1 << 14) -> np.ndarray:
    """N(0,1) draw rounded to storage, generated in chunks along axis 0 to bound peak memory."""
    shape = tuple(int(v) for v in shape)
    out = np.empty(shape, dtype=np.uint16 if dtype == "bf16" else np.float32)
    if out.size == 0:
        return out
    n0 = shape[0]
    inner = int(np.prod(shape[1:])) if len(shape) > 1 else 1
    step = max(1, (chunk_rows * 2048) // max(inner, 1))
    for a in range(0, n0, step):
        b = min(n0, a + step)
        blk = rng.standard_normal((b - a,) + shape[1:], dtype=np.float32)
        out[a:b] = to_storage(blk, dtype)
    return out


# --------------------------------------------------------------------------- workload record
@dataclass
class AttnWorkload:
    """One batch for kv_append + attn_prefixed (all arrays host-side, storage dtype)."""

    name: str
    dtype: str
    num_q_heads: int
    num_kv_heads: int
    head_dim: int
    prefix_len: np.ndarray  # [B] int32
    q_len: np.ndarray  # [B] int32
    cu_q: np.ndarray  # [B+1] int32
    page_table: np.ndarray  # [B, max_pages] int32 (unused entries = -1)
    num_pages: int
    k_pool: np.ndarray  # [num_pages, Hkv, 16, d] storage; holds the cached prefixes
    v_pool: np.ndarray
    q_block: np.ndarray  # [total_q, Hq, d] storage
    k_new: np.ndarray  # [total_q, Hkv, d] storage
    v_new: np.ndarray
    notes: dict = field(default_factory=dict)

    @property
    def batch(self) -> int:
        return int(self.prefix_len.shape[0])

    @property
    def total_q(self) -> int:
        return int(self.cu_q[-1])

    @property
    def group(self) -> int:
        return self.num_q_heads // self.num_kv_heads


@dataclass
class AcceptWorkload:
    """Logits and drafts for the greedy-accept step."""

    name: str
    dtype: str
    vocab: int
    row_stride: int
    logits: np.ndarray  # [rows, row_stride] storage
    drafts: np.ndarray  # [rows - B] int32
    cu_q: np.ndarray  # [B+1] int32
    prefix_len: np.ndarray  # [B] int32
    planted_targets: Optional[np.ndarray] = None  # [rows] int32 when logits were planted
    planned_accept: Optional[np.ndarray] = None  # [B] int32 when drafts follow a plan


def cu_from_q(q_len) -> np.ndarray:
    q_len = np.asarray(q_len, dtype=np.int64)
    cu = np.zeros(q_len.shape[0] + 1, dtype=np.int32)
    cu[1:] = np.cumsum(q_len)
    return cu


def pages_needed(n_tokens: int) -> int:
    return (int(n_tokens) + PAGE - 1) // PAGE


# --------------------------------------------------------------------------- layout helpers
def gather_contiguous(pool: np.ndarray, page_row: np.ndarray, length: int) -> np.ndarray:
    """Copy the first ``length`` tokens of one sequence out of a paged pool: ``[length, Hkv, d]``.

    Pure index gather (layout only).
    """
    npg = pages_needed(length)
    pages = pool[np.asarray(page_row[:npg], dtype=np.int64)]  # [npg, Hkv, 16, d]
    seq = np.transpose(pages, (0, 2, 1, 3)).reshape(npg * PAGE, pool.shape[1], pool.shape[3])
    return np.ascontiguousarray(seq[:length])


def scatter_contiguous(pool: np.ndarray, page_row: np.ndarray, start: int, rows: np.ndarray) -> None:
    """Write ``rows`` (``[n, Hkv, d]``) at token slots ``start..start+n-1`` of one sequence (layout only)."""
    for t in range(rows.shape[0]):
        tok = start + t
        pool[int(page_row[tok // PAGE]), :, tok % PAGE, :] = rows[t]


def build_page_table(rng: np.random.Generator, lengths_total, shared_prefix_tokens: int = 0,
                     spare_pages: int = 0):
    """Assign physical pages to sequences by a seeded permutation.

    ``lengths_total[s]`` is the token capacity sequence ``s`` needs (prefix + block).  The first
    ``shared_prefix_tokens`` tokens (a multiple of 16) map to the same physical pages in every
    sequence; the rest are private.  Returns ``(page_table[B, max_pages], num_pages)``.
    """
    lengths_total = [int(v) for v in lengths_total]
    assert shared_prefix_tokens % PAGE == 0
    n_shared = shared_prefix_tokens // PAGE
    per_seq = [pages_needed(L) for L in lengths_total]
    for n in per_seq:
        assert n >= n_shared, "every sequence must contain the shared prefix"
    n_private = sum(n - n_shared for n in per_seq)
    num_pages = n_shared + n_private + int(spare_pages)
    perm = rng.permutation(num_pages).astype(np.int32)
    max_pages = max(per_seq) if per_seq else 0
    table = np.full((len(per_seq), max_pages), -1, dtype=np.int32)
    shared = perm[:n_shared]
    cursor = n_shared
    for s, n in enumerate(per_seq):
        table[s, :n_shared] = shared
        k = n - n_shared
        table[s, n_shared:n] = perm[cursor:cursor + k]
        cursor += k
    return table, num_pages


def make_attn_workload(name: str, seed: int, dtype: str, num_q_heads: int, num_kv_heads: int,
                       head_dim: int, prefix_len, q_len, shared_prefix_tokens: int = 0,
                       spare_pages: int = 0, notes: Optional[dict] = None) -> AttnWorkload:
    """Draw one batch: a pool whose every slot is N(0,1) (so the cached prefixes are whatever the
    page table points at), plus the block's Q / K_new / V_new."""
    rng = np.random.default_rng(seed)
    prefix_len = np.asarray(prefix_len, dtype=np.int32)
    q_len = np.asarray(q_len, dtype=np.int32)
    cu_q = cu_from_q(q_len)
    total_q = int(cu_q[-1])
    table, num_pages = build_page_table(rng, prefix_len.astype(np.int64) + q_len.astype(np.int64),
                                        shared_prefix_tokens, spare_pages)
    k_pool = _normal_storage(rng, (num_pages, num_kv_heads, PAGE, head_dim), dtype)
    v_pool = _normal_storage(rng, (num_pages, num_kv_heads, PAGE, head_dim), dtype)
    q_block = _normal_storage(rng, (total_q, num_q_heads, head_dim), dtype)
    k_new = _normal_storage(rng, (total_q, num_kv_heads, head_dim), dtype)
    v_new = _normal_storage(rng, (total_q, num_kv_heads, head_dim), dtype)
    return AttnWorkload(name, dtype, num_q_heads, num_kv_heads, head_dim, prefix_len, q_len, cu_q,
                        table, num_pages, k_pool, v_pool, q_block, k_new, v_new, notes or {})


# --------------------------------------------------------------------------- accept inputs
def natural_logits(seed: int, rows: int, vocab: int, dtype: str, row_stride: Optional[int] = None) -> np.ndarray:
    """N(0,1) logits rounded to storage; columns beyond ``vocab`` (row padding) hold +8 so that a
    reader that ignores ``vocab`` is caught."""
    rng = np.random.default_rng(seed)
    row_stride = int(row_stride or vocab)
    x = np.full((rows, row_stride), 8.0, dtype=np.float32)
    x[:, :vocab] = rng.standard_normal((rows, vocab), dtype=np.float32)
    return to_storage(x, dtype)


def plant_targets(logits: np.ndarray, dtype: str, targets: np.ndarray, value: float = 8.0) -> None:
    """Overwrite ``logits[r, targets[r]]`` with ``value`` (exactly representable, far above any
    N(0,1) draw) so the winning index of every row is known without computing it."""
    v = to_storage(np.asarray([value], dtype=np.float32), dtype)[0]
    logits[np.arange(logits.shape[0]), np.asarray(targets, dtype=np.int64)] = v


def make_drafts(seed: int, targets: np.ndarray, cu_q: np.ndarray, planned_accept: np.ndarray,
                vocab: int) -> np.ndarray:
    """Build drafts so that exactly ``planned_accept[s]`` leading drafts of sequence ``s`` equal the
    per-row target of the previous row.  Draft ``a+1`` is a guaranteed mismatch, draft ``a+2`` is
    planted equal to its row's target (a coincidental later match that must not count), the rest
    are random tokens.  ``targets[r]`` is the winning token of logits row ``r``.
    """
    rng = np.random.default_rng(seed)
    B = len(cu_q) - 1
    out = np.zeros(int(cu_q[-1]) - B, dtype=np.int32)
    for s in range(B):
        r0, r1 = int(cu_q[s]), int(cu_q[s + 1])
        k = r1 - r0 - 1
        a = int(planned_accept[s])
        assert 0 <= a <= k
        base = r0 - s
        for i in range(1, k + 1):  # draft i is checked against the target of row i-1
            t_prev = int(targets[r0 + i - 1])
            if i <= a:
                d = t_prev
            elif i == a + 1:
                d = (t_prev + 1 + int(rng.integers(0, vocab - 1))) % vocab
            elif i == a + 2:
                d = t_prev
            else:
                d = int(rng.integers(0, vocab))
            out[base + i - 1] = d
    return out


def make_planted_accept(name: str, seed: int, dtype: str, vocab: int, q_len, prefix_len,
                        planned_accept=None, row_stride: Optional[int] = None) -> AcceptWorkload:
    """Logits with a planted winner per row and drafts following an accept-length plan (uniform over
    0..k when ``planned_accept`` is None)."""
    rng = np.random.default_rng(seed)
    q_len = np.asarray(q_len, dtype=np.int32)
    cu_q = cu_from_q(q_len)
    rows = int(cu_q[-1])
    logits = natural_logits(seed + 1000003, rows, vocab, dtype, row_stride)
    targets = rng.integers(0, vocab, size=rows).astype(np.int32)
    plant_targets(logits, dtype, targets)
    if planned_accept is None:
        planned_accept = np.array([int(rng.integers(0, int(q))) for q in q_len], dtype=np.int32)
    planned_accept = np.asarray(planned_accept, dtype=np.int32)
    drafts = make_drafts(seed + 7, targets, cu_q, planned_accept, vocab)
    return AcceptWorkload(name, dtype, vocab, int(row_stride or vocab), logits, drafts, cu_q,
                          np.asarray(prefix_len, dtype=np.int32), targets, planned_accept)


# --------------------------------------------------------------------------- the five configs
def c1_tiny_verify() -> AttnWorkload:
    """1 sequence, prefix 256 + q=4, 4/2 heads, d=64, fp32, 17 pages inside a 64-page pool."""
    return make_attn_workload("c1_tiny_verify", 1, "f32", 4, 2, 64, [256], [4], spare_pages=64 - 17)


def c2_decode_verify(seed: int = 2, dtype: str = "bf16") -> AttnWorkload:
    """Batch 1, cached context 4096, q=8 (7 drafts + the last emitted token), GQA 32/8, d=128."""
    return make_attn_workload("c2_decode_verify", seed, dtype, 32, 8, 128, [4096], [8], spare_pages=7)


def c3_prefix_prefill(seed: int = 3) -> AttnWorkload:
    """Batch 1, cached prefix 3072 + uncached suffix 512, GQA 24/8, d=128."""
    return make_attn_workload("c3_prefix_prefill", seed, "bf16", 24, 8, 128, [3072], [512])


def c4_lengths(seed: int = 4):
    """Lengths of the ragged mixed batch: lognormal prefixes (median 4096, sigma 0.75, clipped to
    1024..16384, then raised to >= 2048 so each sequence contains the shared 2048 tokens);
    sequences 0..7 carry verify blocks, 8..15 suffix prefill."""
    rng = np.random.default_rng(seed)
    P = np.clip(np.exp(rng.normal(np.log(4096.0), 0.75, size=16)), 1024, 16384).astype(np.int64)
    P = np.maximum(P, 2048)
    q = np.empty(16, dtype=np.int64)
    q[:8] = rng.choice([1, 2, 4, 8, 16], size=8)
    q[8:] = rng.integers(128, 1025, size=8)
    return P.astype(np.int32), q.astype(np.int32)


def c4_ragged_mixed(seed: int = 4) -> AttnWorkload:
    P, q = c4_lengths(seed)
    return make_attn_workload("c4_ragged_mixed", seed + 100, "bf16", 32, 8, 128, P, q,
                              shared_prefix_tokens=2048)


def c5_long_context(seed: int = 5, verify_only: bool = False, prefill_only: bool = False) -> AttnWorkload:
    """4 x (P=32768, q=8) plus 1 x (P=30720, q=2048); GQA 32/8, d=128."""
    P = [32768] * 4 + [30720]
    q = [8] * 4 + [2048]
    if verify_only:
        P, q = P[:4], q[:4]
    if prefill_only:
        P, q = P[4:], q[4:]
    return make_attn_workload("c5_long_context", seed, "bf16", 32, 8, 128, P, q)

