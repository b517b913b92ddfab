"""GPU parity: the CUDA path (through the C ABI) against the CPU oracle on the same seeded inputs.

Attention: max-abs error <= 1e-2 and per-(row, head) normwise relative error <= 2e-2.
KV append, argmax, accept lengths, next tokens, committed lengths: bit-exact.
"""
import numpy as np
import pytest
import torch

import oracle
from paper_2605_10380_b200 import agx
from paper_2605_10380_b200 import workloads as W
from tests.gpu_util import (DeviceBatch, check_attention, dev, host_storage, oracle_pools_after_append,
                            run_accept)

pytestmark = pytest.mark.gpu


def run_and_check(w, sample=None, poison=False, strict=False, fused=False, select=None, options=()):
    """sample=(seed, n): n random (row, head) pairs per sequence plus the corners; select={s: (rows, heads)}: those
    pairs for sequence s and EVERY output row of the other sequences; neither: every output row of the batch."""
    b = DeviceBatch(w)
    for opt, val in options:
        b.h.set_option(opt, val)
    if poison:  # slots past P + q in every sequence's last page hold NaN: they must never be read
        nanbits = 0x7FC0 if w.dtype == "bf16" else np.float32(np.nan)
        for s in range(w.batch):
            L = int(w.prefix_len[s] + w.q_len[s])
            if L % 16:
                pg = int(w.page_table[s, L // 16])
                kp = host_storage(b.k_pool, w.dtype); vp = host_storage(b.v_pool, w.dtype)
                kp[pg, :, L % 16:, :] = nanbits; vp[pg, :, L % 16:, :] = nanbits
                b.k_pool.copy_(dev(kp, w.dtype)); b.v_pool.copy_(dev(vp, w.dtype))
    if fused:
        out, lse = b.attend_append()
    else:
        b.append()
        out, lse = b.attend()
    assert b.status() == 0
    kp, vp = oracle_pools_after_append(w)
    # append parity, bit-exact on the touched pages
    gk = host_storage(b.k_pool, w.dtype); gv = host_storage(b.v_pool, w.dtype)
    if not poison:
        assert np.array_equal(gk, kp) and np.array_equal(gv, vp)
    if sample is None and select is None:
        ref, ref_lse = oracle.attn_paged_batch(w.q_block, kp, vp, w.page_table, w.dtype, w.prefix_len, w.q_len, w.cu_q)
        stats = check_attention(out, ref, w.name, strict)
        assert np.max(np.abs(lse - ref_lse)) <= 2e-3, "lse"
    elif select is not None:
        stats = (0.0, 0.0)
        for s in range(w.batch):
            q = int(w.q_len[s]); r0 = int(w.cu_q[s])
            if s in select:
                si, sh = (np.asarray(a, dtype=np.int32) for a in select[s])
                ref, ref_lse, _ = oracle.attn_paged(w.q_block[r0:r0 + q], kp, vp, w.page_table[s], w.dtype,
                                                    int(w.prefix_len[s]), select=(si, sh))
                got, got_lse = out[r0 + si, sh], lse[r0 + si, sh]
            else:
                ref, ref_lse, _ = oracle.attn_paged(w.q_block[r0:r0 + q], kp, vp, w.page_table[s], w.dtype, int(w.prefix_len[s]))
                got, got_lse = out[r0:r0 + q], lse[r0:r0 + q]
            st = check_attention(got, ref, f"{w.name} seq {s}", strict)
            stats = (max(stats[0], st[0]), max(stats[1], st[1]))
            assert np.max(np.abs(got_lse - ref_lse)) <= 2e-3
    else:
        rng = np.random.default_rng(sample[0])
        stats = (0.0, 0.0)
        for s in range(w.batch):
            q = int(w.q_len[s]); r0 = int(w.cu_q[s])
            n = min(sample[1], q * w.num_q_heads)
            si = np.concatenate([[0, q - 1], rng.integers(0, q, n)]).astype(np.int32)
            sh = np.concatenate([[0, w.num_q_heads - 1], rng.integers(0, w.num_q_heads, n)]).astype(np.int32)
            ref, ref_lse, _ = oracle.attn_paged(w.q_block[r0:r0 + q], kp, vp, w.page_table[s], w.dtype,
                                                int(w.prefix_len[s]), select=(si, sh))
            st = check_attention(out[r0 + si, sh], ref, f"{w.name} seq {s}", strict)
            stats = (max(stats[0], st[0]), max(stats[1], st[1]))
            assert np.max(np.abs(lse[r0 + si, sh] - ref_lse)) <= 2e-3
    return b, stats


# ------------------------------------------------------------------ named configurations
def test_c1_tiny_verify_fp32():
    b, _ = run_and_check(W.c1_tiny_verify(), strict=True)
    assert b.launches >= 1


def test_c1_tiny_verify_bf16_rounded_inputs_d128():
    w = W.make_attn_workload("c1_bf16", 1, "bf16", 4, 2, 128, [256], [4], spare_pages=47)
    run_and_check(w)


def test_c1_tiny_verify_bf16_head_dim_64():
    """The tiny configuration's own shape (4/2 heads, d = 64, P = 256, q = 4) with bf16 storage, and two more shapes of
    the scalar kernel that serves bf16 pools with head_dim 64: every output row, both call forms."""
    w = W.make_attn_workload("c1_bf16_d64", 1, "bf16", 4, 2, 64, [256], [4], spare_pages=47)
    run_and_check(w, strict=True)
    w2 = W.make_attn_workload("bf16_d64_ragged", 12, "bf16", 8, 2, 64, [1000, 37, 0], [5, 40, 17])
    run_and_check(w2, poison=True)
    run_and_check(w2, poison=True, fused=True)


def test_c2_decode_verify():
    b, stats = run_and_check(W.c2_decode_verify(), strict=True)
    assert b.ws_bytes > 0  # the context is split over many CTAs


def test_c2_accept_bf16_uniform_accept_lengths():
    h = agx.Handle(32, 8, 128, "bf16")
    for a in range(8):
        aw = W.make_planted_accept("c2_accept", 200 + a, "bf16", 128256, [8], [4096], planned_accept=[a])
        ref = oracle.accept_greedy(aw.logits, "bf16", aw.vocab, aw.drafts, aw.cu_q, aw.prefix_len)
        got = run_accept(h, aw)
        for g, r in zip(got, ref):
            assert np.array_equal(g, r)
        assert got[1][0] == a and got[3][0] == 4096 + a + 1


def test_c1_accept_fp32_first_two_of_three_match():
    logits = W.natural_logits(1, 4, 1024, "f32")
    am, _, _, _ = oracle.accept_greedy(logits, "f32", 1024, np.zeros(0, np.int32), np.arange(5, dtype=np.int32),
                                       np.zeros(4, np.int32))
    drafts = np.array([am[0], am[1], (am[2] + 1) % 1024], dtype=np.int32)  # first 2 of 3 match
    aw = W.AcceptWorkload("c1_accept", "f32", 1024, 1024, logits, drafts, np.array([0, 4], np.int32),
                          np.array([256], np.int32))
    h = agx.Handle(4, 2, 64, "f32")
    got = run_accept(h, aw)
    ref = oracle.accept_greedy(logits, "f32", 1024, drafts, aw.cu_q, aw.prefix_len)
    for g, r in zip(got, ref):
        assert np.array_equal(g, r)
    assert got[1][0] == 2 and got[2][0] == am[2] and got[3][0] == 259


def test_c4_ragged_mixed_batch_shared_prefix():
    """16 sequences, lognormal prefixes, verify blocks and suffix prefills in one call, first 2048
    tokens' pages shared by all: EVERY output row of every sequence against the oracle."""
    w = W.c4_ragged_mixed()
    assert np.all(w.page_table[:, :128] == w.page_table[0, :128])
    b, _ = run_and_check(w, strict=True)
    assert b.launches >= 3  # split-KV kernel(s), tile kernel, combine


def tile_edge_rows(q, G, hq, seed, extra):
    """(row, head) pairs that look into every CTA of the 256-row schedule: for every KV head the rows at
    positions 0, 127, 128 and 255 of every 256-row chunk (first and last row of both Q tiles), plus `extra`
    seeded random pairs."""
    hkv = hq // G
    si, sh = [], []
    for g in range(hkv):
        for r in range(0, q * G):
            if r % 256 in (0, 127, 128, 255) or r == q * G - 1:
                si.append(r // G); sh.append(g * G + r % G)
    rng = np.random.default_rng(seed)
    si += rng.integers(0, q, extra).tolist(); sh += rng.integers(0, hq, extra).tolist()
    return np.asarray(si, np.int32), np.asarray(sh, np.int32)


def test_c5_long_context_verify_and_prefill():
    """4 x (P = 32768, q = 8) plus 1 x (P = 30720, q = 2048) in one call.  Every output row of the four verify
    blocks is compared with the oracle; of the 2048-row prefill, the first and last row of every 128-row Q tile
    of every KV head (so every (row chunk, KV head, KV split) CTA is looked at) plus 200 random (row, head)
    pairs.  Then the accept step on bf16 logits [4 x 8, 128256]."""
    w = W.c5_long_context()
    b, _ = run_and_check(w, strict=True, select={4: tile_edge_rows(2048, 4, 32, 6, 200)})
    h = agx.Handle(32, 8, 128, "bf16")
    aw = W.make_planted_accept("c5_accept", 55, "bf16", 128256, [8] * 4, [32768] * 4)
    ref = oracle.accept_greedy(aw.logits, "bf16", aw.vocab, aw.drafts, aw.cu_q, aw.prefix_len)
    got = run_accept(h, aw)
    for g, r in zip(got, ref):
        assert np.array_equal(g, r)
    assert np.array_equal(got[1], aw.planned_accept)


# ------------------------------------------------------------------ small-q kernel: shapes and edges
@pytest.mark.parametrize("P,q,hq,hkv", [
    (0, 1, 32, 8), (1, 1, 32, 8), (15, 1, 8, 8), (16, 2, 32, 8), (17, 4, 32, 8), (63, 8, 32, 8), (64, 8, 32, 8),
    (65, 16, 32, 8), (1000, 3, 24, 8), (2049, 5, 32, 8), (5000, 8, 32, 8), (777, 16, 32, 8), (300, 7, 4, 1),
    (130, 1, 4, 4), (4095, 2, 16, 2),
])
def test_small_q_shapes(P, q, hq, hkv):
    w = W.make_attn_workload(f"small_{P}_{q}", 1000 + P + q, "bf16", hq, hkv, 128, [P], [q], spare_pages=3)
    run_and_check(w, poison=True)


@pytest.mark.parametrize("merge", ["clusters", "combine_kernel"])
@pytest.mark.parametrize("P,q,hq,hkv,batch", [
    (4096, 8, 32, 8, 1),      # 17 splits squeezed into clusters of 16 where eight such clusters fit the device
    (4096, 1, 32, 8, 1), (3000, 5, 32, 8, 1), (700, 8, 32, 8, 1), (300, 2, 32, 8, 1), (1000, 3, 24, 8, 1),
    (6000, 7, 8, 8, 1), (2500, 12, 4, 1, 1), (4090, 16, 32, 8, 1),
    (4096, 8, 32, 8, 4),      # four equal sequences: clusters of 4
    (2000, 4, 32, 8, 2),
])
def test_small_q_split_merge_in_clusters_and_by_combine_kernel(P, q, hq, hkv, batch, merge, monkeypatch):
    """The KV splits of the warp-MMA kernel merged through the clusters' shared memory (one launch) and through
    partials in global memory plus the combine kernel (two launches): both against the oracle."""
    monkeypatch.setenv("AGX_CLUSTER_MERGE", "1" if merge == "clusters" else "0")
    w = W.make_attn_workload(f"cl_{P}_{q}_{batch}", 500 + P + q, "bf16", hq, hkv, 128, [P + 16 * i for i in range(batch)] if batch == 2 else [P] * batch,
                             [q] * batch, spare_pages=2)
    b, _ = run_and_check(w, poison=True, sample=(5, 24) if batch > 1 else None)
    if merge == "clusters" and batch == 1 and 700 <= P <= 1000:     # clusters of 3 or 4 fit any device; one launch, no combine
        assert b.launches == 1
    if merge == "combine_kernel" and P >= 700:
        assert b.launches == 2


@pytest.mark.parametrize("P,q,hq,hkv", [(0, 1, 32, 8), (17, 4, 32, 8), (1000, 3, 24, 8), (2049, 5, 32, 8), (4096, 8, 32, 8), (300, 16, 4, 4)])
def test_small_q_kernel_with_four_kv_groups(P, q, hq, hkv, monkeypatch):
    """AGX_SMALL_KW=4: four pages per pipeline stage, each warp owning two 16-column groups of O."""
    monkeypatch.setenv("AGX_SMALL_KW", "4")
    w = W.make_attn_workload(f"kw4_{P}_{q}", 900 + P + q, "bf16", hq, hkv, 128, [P], [q], spare_pages=2)
    run_and_check(w, poison=True)


@pytest.mark.parametrize("P,q", [
    ([2100, 2048, 2300, 1990], [8, 8, 1, 5]),          # > 8k tokens in all: warp-MMA kernel with 4-page stages
    ([9000, 8200, 8192, 7000], [4, 8, 8, 1]),          # > 24k tokens in all: every block on the stream schedule
    ([3000, 100], [8, 8]), ([5000, 4000, 17], [1, 1, 1]),
    ([8192, 8192], [8, 8]),      # stream schedule whose last KV split is one short tile: its CTAs reach the epilogue at once
])
def test_batches_dispatched_by_their_total_context(P, q):
    w = W.make_attn_workload(f"batch_{sum(P)}", 4000 + sum(P), "bf16", 32, 8, 128, P, q, spare_pages=2)
    run_and_check(w, sample=(9, 20), poison=True)
    run_and_check(w, sample=(9, 20), fused=True)


@pytest.mark.parametrize("fused", [False, True])
def test_more_sequences_than_one_launch_holds(fused):
    """70 sequences (a launch holds 48): several launches per kernel kind, contexts from empty to a few pages, one long."""
    rng = np.random.default_rng(123)
    P = rng.integers(0, 300, 70).tolist(); P[5] = 0; P[17] = 5000; P[40] = 2049
    q = rng.integers(1, 9, 70).tolist(); q[17] = 3; q[33] = 40       # one block of 160 rows rides along
    w = W.make_attn_workload("many_seqs", 321, "bf16", 32, 8, 128, P, q, spare_pages=1)
    run_and_check(w, poison=not fused, fused=fused)


@pytest.mark.parametrize("hq,hkv", [(16, 2), (16, 16), (8, 1), (40, 8)])
def test_other_head_layouts(hq, hkv):
    G = hq // hkv
    P = [1000, 37, 4100, 0]
    q = [max(1, 32 // G), 1, max(1, 16 // G), 2]
    w = W.make_attn_workload(f"heads_{hq}_{hkv}", 55 + hq, "bf16", hq, hkv, 128, P, q, spare_pages=1)
    run_and_check(w, poison=True)
    run_and_check(w, fused=True)


@pytest.mark.parametrize("seed", [1, 2, 3])
def test_random_batches_against_oracle(seed):
    """Ten random batches per seed: 1-6 sequences, contexts from empty to ~20k tokens (skewed to short), verify-sized
    blocks with an occasional long one; sampled rows against the oracle, fused and unfused."""
    rng = np.random.default_rng(1000 + seed)
    for case in range(10):
        B = int(rng.integers(1, 7))
        P = [int(x) for x in np.minimum(rng.exponential(3000, B).astype(np.int64) * int(rng.integers(1, 4)), 20000)]
        q = [int(rng.integers(1, 17)) if rng.random() < 0.85 else int(rng.integers(17, 300)) for _ in range(B)]
        if rng.random() < 0.3:
            P[0] = int(rng.integers(0, 3)) * 4096      # page- and tile-aligned prefixes, empty ones
        w = W.make_attn_workload(f"rand_{seed}_{case}", 9000 + 100 * seed + case, "bf16", 32, 8, 128, P, q, spare_pages=1)
        run_and_check(w, sample=(case, 12), fused=bool(case & 1))


def test_sixty_random_batches_fused_call_bit_identical_and_reproducible():
    """Random head layouts, 1-8 sequences, contexts to 24k tokens, blocks from 1 to 700 rows, all in one process (kernel
    kinds follow one another in every order): the fused call leaves the pools and the output bit-identical to append +
    attention, twice over, with a clean status word."""
    rng = np.random.default_rng(77)
    heads = [(32, 8), (32, 8), (24, 8), (16, 2), (8, 8), (40, 8)]
    for case in range(60):
        hq, hkv = heads[int(rng.integers(0, len(heads)))]
        B = int(rng.integers(1, 9))
        scale = [300, 3000, 9000][int(rng.integers(0, 3))]
        P = [int(min(x, 24000)) for x in rng.exponential(scale, B)]
        if rng.random() < 0.3:
            P[int(rng.integers(0, B))] = int(rng.integers(0, 6)) * 2048
        q = []
        for _ in range(B):
            u = rng.random()
            q.append(int(rng.integers(1, 17)) if u < 0.8 else int(rng.integers(17, 140)) if u < 0.95 else int(rng.integers(140, 700)))
        w = W.make_attn_workload(f"rnd_{case}", 50000 + case, "bf16", hq, hkv, 128, P, q, spare_pages=1)
        two = DeviceBatch(w); two.append(); two.attend()
        one = DeviceBatch(w); one.attend_append()
        again = DeviceBatch(w); again.attend_append()
        assert one.status() == 0 and two.status() == 0 and again.status() == 0, (case, P, q)
        assert torch.equal(one.k_pool, two.k_pool) and torch.equal(one.v_pool, two.v_pool), (case, P, q)
        assert torch.equal(one.out, two.out) and torch.equal(one.out, again.out), (case, P, q)
        assert bool(torch.isfinite(one.out.float()).all()), (case, P, q)


def test_small_q_ragged_batch_with_shared_prefix():
    P = [2048, 2100, 4000, 2048 + 15, 9000, 2500, 3001, 2048]
    q = [1, 2, 4, 8, 16, 3, 5, 8]
    w = W.make_attn_workload("ragged_small", 42, "bf16", 32, 8, 128, P, q, shared_prefix_tokens=2048)
    run_and_check(w, sample=(7, 12))


def test_q1_equals_plain_decode_on_gpu():
    w = W.make_attn_workload("decode", 9, "bf16", 32, 8, 128, [1234], [1])
    b = DeviceBatch(w); b.append(); out, _ = b.attend()
    kp, vp = oracle_pools_after_append(w)
    K = W.gather_contiguous(kp, w.page_table[0], 1235); V = W.gather_contiguous(vp, w.page_table[0], 1235)
    ref = oracle.decode_plain(w.q_block[0], K, V, "bf16")
    check_attention(out[0], ref, "decode")


def test_split_results_are_bit_reproducible():
    w = W.c2_decode_verify(seed=12)
    b = DeviceBatch(w); b.append()
    a, _ = b.attend()
    b.out.zero_()
    c, _ = b.attend()
    assert np.array_equal(a, c)


def test_fp32_path_shapes():
    for (P, q, hq, hkv, d) in [(0, 1, 4, 2, 64), (100, 5, 4, 2, 64), (700, 3, 8, 2, 128), (31, 20, 4, 4, 64)]:
        w = W.make_attn_workload(f"f32_{P}_{q}", 5 + P, "f32", hq, hkv, d, [P, P + 3], [q, 1], spare_pages=2)
        run_and_check(w, poison=True)


def test_mma_sync_kernel_handles_large_q(monkeypatch):
    """The warp-MMA kernel also serves long blocks (row chunks); it is the baseline the tensor-core
    tile kernel is measured against."""
    monkeypatch.setenv("AGX_FORCE_MMA_SYNC", "1")
    w = W.make_attn_workload("mma_large", 77, "bf16", 24, 8, 128, [500, 37], [200, 130])
    run_and_check(w, sample=(3, 40))


# ------------------------------------------------------------------ KV append alone
def test_kv_append_ragged_bit_exact_and_untouched_elsewhere():
    w = W.make_attn_workload("append", 5, "bf16", 32, 8, 128, [5, 30, 16, 0, 4095], [3, 1, 20, 17, 600], spare_pages=5)
    b = DeviceBatch(w); b.append(); torch.cuda.synchronize()
    kp, vp = oracle_pools_after_append(w)
    assert np.array_equal(host_storage(b.k_pool, "bf16"), kp)
    assert np.array_equal(host_storage(b.v_pool, "bf16"), vp)


def test_bad_page_id_sets_status_and_does_not_fault():
    w = W.make_attn_workload("badpage", 6, "bf16", 32, 8, 128, [100], [4])
    w.page_table[0, 2] = w.num_pages + 1000
    b = DeviceBatch(w); b.append(); b.attend()
    assert b.status() & agx.AGX_DEV_BAD_PAGE
    assert b.status() == 0  # cleared by the read


# ------------------------------------------------------------------ accept
def test_accept_natural_ties_and_special_values():
    h = agx.Handle(32, 8, 128, "bf16")
    x = W.natural_logits(5, 40, 128256, "bf16")
    am_ref, _, _, _ = oracle.accept_greedy(x, "bf16", 128256, np.zeros(0, np.int32), np.arange(41, dtype=np.int32),
                                           np.zeros(40, np.int32))
    q_len = [8, 1, 16, 4, 2, 9]
    cu = W.cu_from_q(q_len)
    rng = np.random.default_rng(0)
    plan = np.array([int(rng.integers(0, q)) for q in q_len], dtype=np.int32)
    drafts = W.make_drafts(3, am_ref, cu, plan, 128256)
    aw = W.AcceptWorkload("ties", "bf16", 128256, 128256, x, drafts, cu, np.arange(6, dtype=np.int32) * 100)
    got = run_accept(h, aw)
    ref = oracle.accept_greedy(x, "bf16", 128256, drafts, cu, aw.prefix_len)
    for g, r in zip(got, ref):
        assert np.array_equal(g, r)
    assert np.array_equal(got[1], plan)


@pytest.mark.parametrize("dtype", ["f32", "bf16"])
def test_accept_special_values_padding_and_odd_vocab(dtype):
    V, stride = 1001, 1008
    x = np.full((6, stride), 9.0, dtype=np.float32)
    x[:, :V] = -1.0
    x[0, [3, 700]] = 2.0
    x[1, :V] = -0.0; x[1, 5] = 0.0
    x[2, :V] = np.nan; x[2, 999] = -50.0
    x[3, :V] = np.nan
    x[4, :V] = -np.inf
    x[5, 1000] = np.inf; x[5, 1] = 1e30
    xs = W.to_storage(x, dtype)
    cu = np.arange(7, dtype=np.int32)
    aw = W.AcceptWorkload("special", dtype, V, stride, xs, np.zeros(0, np.int32), cu, np.zeros(6, np.int32))
    h = agx.Handle(4, 2, 64, "f32")
    got = run_accept(h, aw)
    ref = oracle.accept_greedy(xs, dtype, V, aw.drafts, cu, aw.prefix_len)
    assert got[0].tolist() == [3, 0, 999, 0, 0, 1000]
    for g, r in zip(got, ref):
        assert np.array_equal(g, r)


def test_accept_many_rows_and_unaligned_rows():
    h = agx.Handle(4, 2, 64, "f32")
    aw = W.make_planted_accept("many", 31, "bf16", 3001, [5] * 60 + [1] * 40, np.arange(100), row_stride=3001)
    got = run_accept(h, aw)
    ref = oracle.accept_greedy(aw.logits, "bf16", aw.vocab, aw.drafts, aw.cu_q, aw.prefix_len)
    for g, r in zip(got, ref):
        assert np.array_equal(g, r)
    # twice in a row on the same handle: the ticket counter resets itself
    got2 = run_accept(h, aw)
    for g, r in zip(got2, ref):
        assert np.array_equal(g, r)


# ------------------------------------------------------------------ invariants of the definition, on the GPU
def _attend(w):
    b = DeviceBatch(w); b.append(); out, lse = b.attend()
    assert b.status() == 0
    return out, lse


@pytest.mark.parametrize("P,q", [(700, 8), (9000, 8), (1500, 200)])
def test_gpu_output_is_unchanged_by_a_joint_permutation_of_the_cached_prefix(P, q):
    """No positional term inside the library: shuffling the cached prefix's (K, V) tokens together leaves every
    output row unchanged up to summation order (small-q, stream and tile kernels)."""
    w = W.make_attn_workload("perm", 71, "bf16", 32, 8, 128, [P], [q])
    a, lse_a = _attend(w)
    K = W.gather_contiguous(w.k_pool, w.page_table[0], P); V = W.gather_contiguous(w.v_pool, w.page_table[0], P)
    perm = np.random.default_rng(5).permutation(P)
    w2 = W.make_attn_workload("perm", 71, "bf16", 32, 8, 128, [P], [q])
    W.scatter_contiguous(w2.k_pool, w2.page_table[0], 0, K[perm]); W.scatter_contiguous(w2.v_pool, w2.page_table[0], 0, V[perm])
    b, lse_b = _attend(w2)
    assert np.max(np.abs(a - b)) <= 4e-3 and np.max(np.abs(lse_a - lse_b)) <= 1e-3


def test_gpu_gqa_equals_mha_with_replicated_kv_heads_and_ignores_pages_beyond_the_sequence():
    w = W.make_attn_workload("gqa", 72, "bf16", 8, 2, 128, [1000], [8], spare_pages=9)
    a, _ = _attend(w)
    rep = lambda x: np.repeat(x, 4, axis=1)
    w2 = W.AttnWorkload("mha", "bf16", 8, 8, 128, w.prefix_len, w.q_len, w.cu_q, w.page_table, w.num_pages,
                        rep(w.k_pool), rep(w.v_pool), w.q_block, rep(w.k_new), rep(w.v_new))
    b, _ = _attend(w2)
    assert np.array_equal(a, b)   # same kernel, same per-head arithmetic
    # a longer page table whose extra entries point at pages full of NaN changes nothing
    w3 = W.make_attn_workload("gqa", 72, "bf16", 8, 2, 128, [1000], [8], spare_pages=9)
    table = np.full((1, w3.page_table.shape[1] + 4), -1, dtype=np.int32)
    table[0, :w3.page_table.shape[1]] = w3.page_table[0]
    used = set(w3.page_table[0].tolist())
    spare = [pg for pg in range(w3.num_pages) if pg not in used][:4]
    table[0, w3.page_table.shape[1]:] = spare
    w3.k_pool[spare] = 0x7FC0; w3.v_pool[spare] = 0x7FC0
    w3.page_table = table
    c, _ = _attend(w3)
    assert np.array_equal(a, c)


# ------------------------------------------------------------------ reusing a stored prefix that is cut inside a page
def test_prefix_reuse_with_tail_cut_shares_full_pages_and_copies_the_cut_page():
    """Sec. 4.2: a request matches only the leading part of a stored combination, so the reused KV ends in the
    middle of a page.  The new sequence shares the full pages, gets a private copy of the cut page
    (agx_kv_copy_pages), appends its own block behind the cut, and must see exactly prefix + block; the stored
    sequence's pages are untouched."""
    P_stored, P_cut, q = 200, 37 * 3 + 5, 24            # cut at token 116: 7 full pages shared, page 7 copied
    w = W.make_attn_workload("stored", 81, "bf16", 32, 8, 128, [P_stored], [q], spare_pages=12)
    h = agx.Handle(32, 8, 128, "bf16")
    k_pool, v_pool = dev(w.k_pool, "bf16"), dev(w.v_pool, "bf16")
    k_before = host_storage(k_pool, "bf16").copy()
    stored_row = w.page_table[0]
    used = set(stored_row.tolist())
    fresh = [pg for pg in range(w.num_pages) if pg not in used]
    n_full = P_cut // 16
    new_row = np.full(stored_row.shape[0], -1, dtype=np.int32)
    new_row[:n_full] = stored_row[:n_full]                           # shared, read only
    need = (P_cut + q + 15) // 16 - n_full
    new_row[n_full:n_full + need] = fresh[:need]
    h.kv_copy_pages(k_pool, v_pool, dev(np.array([stored_row[n_full]], np.int32)), dev(np.array([new_row[n_full]], np.int32)))
    table = dev(new_row[None, :].copy())
    h.kv_append(k_pool, v_pool, dev(w.k_new, "bf16"), dev(w.v_new, "bf16"), table, dev(np.array([P_cut], np.int32)),
                dev(np.array([0, q], np.int32)))
    out = torch.zeros((q, 32, 128), dtype=torch.bfloat16, device="cuda")
    Pn, Qn = np.array([P_cut], np.int32), np.array([q], np.int32)
    n = h.attn_workspace_bytes(Pn, Qn)
    ws = torch.empty(max(n, 256), dtype=torch.uint8, device="cuda") if n else None
    h.attn_prefixed(dev(w.q_block, "bf16"), k_pool, v_pool, table, Pn, Qn, out, None, ws)
    torch.cuda.synchronize()
    assert h.get_status() == 0
    # oracle: contiguous K/V = the first P_cut tokens of the stored sequence, then the block
    K = np.concatenate([W.gather_contiguous(w.k_pool, stored_row, P_cut), w.k_new])
    V = np.concatenate([W.gather_contiguous(w.v_pool, stored_row, P_cut), w.v_new])
    ref, _, _ = oracle.attn_contiguous(w.q_block, K, V, "bf16", P_cut)
    check_attention(out.to(torch.float64).cpu().numpy(), ref, "tail cut")
    k_after = host_storage(k_pool, "bf16")
    assert np.array_equal(k_after[stored_row[:(P_stored + 15) // 16]], k_before[stored_row[:(P_stored + 15) // 16]])
    assert np.array_equal(k_after[new_row[n_full], :, :P_cut % 16], k_before[stored_row[n_full], :, :P_cut % 16])
    # bad page ids are flagged, not followed
    h.kv_copy_pages(k_pool, v_pool, dev(np.array([w.num_pages + 3], np.int32)), dev(np.array([0], np.int32)))
    torch.cuda.synchronize()
    assert h.get_status() & agx.AGX_DEV_BAD_PAGE


@pytest.mark.parametrize("zero_copy", ["3", "0"], ids=["read_by_kernel", "staged_copies"])
def test_import_of_stored_pages_from_host_memory_overlapping_attention_on_another_stream(zero_copy, monkeypatch):
    """Stored KV pages (Sec. 4.2) come from pinned host memory into scattered pool pages, bit for bit, on a stream
    of their own while attention over resident pages runs on another; a sequence then attends over the imported
    prefix."""
    monkeypatch.setenv("AGX_ZERO_COPY", zero_copy)
    w = W.make_attn_workload("import", 91, "bf16", 32, 8, 128, [3072], [64], spare_pages=4)
    h = agx.Handle(32, 8, 128, "bf16")
    n_imp = 3072 // 16
    rows = w.page_table[0, :n_imp].astype(np.int64)
    h_k = torch.from_numpy(w.k_pool[rows].copy()).pin_memory(); h_v = torch.from_numpy(w.v_pool[rows].copy()).pin_memory()
    kp, vp = w.k_pool.copy(), w.v_pool.copy()
    kp[rows] = 0; vp[rows] = 0                                       # the pool does not hold the prefix yet
    k_pool, v_pool = dev(kp, "bf16"), dev(vp, "bf16")
    other = DeviceBatch(W.make_attn_workload("busy", 92, "bf16", 32, 8, 128, [20000], [8]))   # resident work for the other stream
    staging = torch.empty(h.kv_import_staging_bytes(n_imp), dtype=torch.uint8, device="cuda")
    dst = dev(w.page_table[0, :n_imp].copy())
    torch.cuda.synchronize()
    side = torch.cuda.Stream()
    with torch.cuda.stream(side):
        h.kv_import_pages(k_pool, v_pool, h_k, h_v, dst, staging, stream=side)
    other.append(); other.attend()                                   # enqueued on the current stream meanwhile
    side.synchronize(); torch.cuda.synchronize()
    assert h.get_status() == 0 and other.status() == 0
    assert np.array_equal(host_storage(k_pool, "bf16"), w.k_pool) and np.array_equal(host_storage(v_pool, "bf16"), w.v_pool)
    b = DeviceBatch(w); b.k_pool, b.v_pool = k_pool, v_pool
    b.append(); out, _ = b.attend()
    kref, vref = oracle_pools_after_append(w)
    rng = np.random.default_rng(1)
    si = rng.integers(0, 64, 30).astype(np.int32); sh = rng.integers(0, 32, 30).astype(np.int32)
    ref, _, _ = oracle.attn_paged(w.q_block, kref, vref, w.page_table[0], "bf16", 3072, select=(si, sh))
    check_attention(out[si, sh], ref, "imported prefix")


# ------------------------------------------------------------------ whole step from host buffers
n_launch = {}


@pytest.mark.parametrize("enqueue_only,memory", [(False, "pinned"), (True, "pinned"), (True, "pageable"), (True, "pinned_copies")])
def test_verify_step_host_matches_oracle(enqueue_only, memory, monkeypatch):
    """Append + attention + accept through the host-buffer entry points (results back in host memory); the enqueue
    variant returns before the work is done and is synchronised by the caller.  Small pinned buffers are read and
    written by the kernels themselves, pageable ones (and pinned ones with AGX_ZERO_COPY=0) go through copies."""
    if memory == "pinned_copies":
        monkeypatch.setenv("AGX_ZERO_COPY", "0")
    w = W.make_attn_workload("host_step", 77, "bf16", 32, 8, 128, [1000, 517, 40], [8, 4, 1], spare_pages=2)
    aw = W.make_planted_accept("host_step_accept", 78, "bf16", 128256, w.q_len, w.prefix_len)
    b = DeviceBatch(w)
    to_t = lambda a, bf: torch.from_numpy(np.ascontiguousarray(a)).view(torch.bfloat16) if bf else torch.from_numpy(np.ascontiguousarray(a))
    pin = lambda a, bf=False: to_t(a, bf).pin_memory() if memory != "pageable" else to_t(a, bf).clone()
    hq, hk, hv = pin(w.q_block, True), pin(w.k_new, True), pin(w.v_new, True)
    hl, hd = pin(aw.logits, True), pin(aw.drafts)
    h_out = torch.zeros((w.total_q, 32, 128), dtype=torch.bfloat16)
    h_out = h_out.pin_memory() if memory != "pageable" else h_out
    h_acc = torch.full((3,), -7, dtype=torch.int32).pin_memory()
    h_nxt = torch.full((3,), -7, dtype=torch.int32).pin_memory()
    h_sl = torch.full((3,), -7, dtype=torch.int32).pin_memory()
    n = b.h.verify_step_host_workspace_bytes(w.prefix_len, w.q_len, "bf16", 128256, 128256)
    ws = torch.empty(n, dtype=torch.uint8, device="cuda")
    b.h.verify_step_host(b.k_pool, b.v_pool, b.page_table, w.prefix_len, w.q_len, hq, hk, hv, hl, "bf16", 128256, 128256,
                         hd, h_out, h_acc, h_nxt, h_sl, ws, enqueue_only=enqueue_only)
    torch.cuda.synchronize()
    assert b.status() == 0
    kp, vp = oracle_pools_after_append(w)
    assert np.array_equal(host_storage(b.k_pool, "bf16"), kp) and np.array_equal(host_storage(b.v_pool, "bf16"), vp)
    ref, _ = oracle.attn_paged_batch(w.q_block, kp, vp, w.page_table, "bf16", w.prefix_len, w.q_len, w.cu_q)
    check_attention(h_out.to(torch.float64).numpy(), ref, "host step")
    n_launch[memory] = b.h.last_launch_count()
    if "pinned" in n_launch and "pinned_copies" in n_launch:      # the kernel that reads the pinned inputs is the one extra launch
        assert n_launch["pinned"] == n_launch["pinned_copies"] + 1
    am, al, nt, sl = oracle.accept_greedy(aw.logits, "bf16", aw.vocab, aw.drafts, aw.cu_q, aw.prefix_len)
    assert np.array_equal(h_acc.numpy(), al) and np.array_equal(h_nxt.numpy(), nt) and np.array_equal(h_sl.numpy(), sl)


@pytest.mark.parametrize("enqueue_only,rows", [(False, None), (True, None), (True, "200"), (True, "0")])
def test_attention_only_host_step_in_row_chunks_matches_oracle(enqueue_only, rows, monkeypatch):
    """A host step that moves several megabytes and has no accept part runs as a pipeline of row chunks (chunked
    prefill: uploads, attention calls and downloads of different chunks overlap on streams of the handle's own).  A
    block long enough to be cut into row chunks with a short last one, a run of two short blocks that share a call and
    a block on its own; default chunk length, a shorter one and the pipeline switched off: the pools and every output
    row against the oracle, and a second step on the same handle right behind the first."""
    if rows is not None:
        monkeypatch.setenv("AGX_HOST_PIPELINE_ROWS", rows)
    w = W.make_attn_workload("host_chunks", 91, "bf16", 32, 8, 128, [600, 333, 50, 700], [1300, 200, 150, 900], spare_pages=2)
    b = DeviceBatch(w)
    to_t = lambda a: torch.from_numpy(np.ascontiguousarray(a)).view(torch.bfloat16).pin_memory()
    hq, hk, hv = to_t(w.q_block), to_t(w.k_new), to_t(w.v_new)
    n = b.h.verify_step_host_workspace_bytes(w.prefix_len, w.q_len, "bf16", 0, 0)
    ws = torch.empty(n, dtype=torch.uint8, device="cuda")
    kp, vp = oracle_pools_after_append(w)
    ref, _ = oracle.attn_paged_batch(w.q_block, kp, vp, w.page_table, "bf16", w.prefix_len, w.q_len, w.cu_q)
    for step in range(2):
        h_out = torch.zeros((w.total_q, 32, 128), dtype=torch.bfloat16).pin_memory()
        b.h.verify_step_host(b.k_pool, b.v_pool, b.page_table, w.prefix_len, w.q_len, hq, hk, hv, None, "bf16", 0, 0,
                             None, h_out, None, None, None, ws, enqueue_only=enqueue_only)
        torch.cuda.synchronize()
        assert b.status() == 0
        assert np.array_equal(host_storage(b.k_pool, "bf16"), kp) and np.array_equal(host_storage(b.v_pool, "bf16"), vp)
        check_attention(h_out.to(torch.float64).numpy(), ref, f"host step in row chunks, step {step}")


def test_verify_step_host_with_more_sequences_than_one_launch_holds():
    """60 sequences through the host-buffer step: lengths travel by copy instead of kernel arguments, attention takes
    several launches."""
    rng = np.random.default_rng(5)
    P = rng.integers(0, 400, 60).tolist(); q = rng.integers(1, 6, 60).tolist()
    w = W.make_attn_workload("host_step_60", 79, "bf16", 32, 8, 128, P, q, spare_pages=1)
    aw = W.make_planted_accept("host_step_60_accept", 80, "bf16", 4099, w.q_len, w.prefix_len)
    b = DeviceBatch(w)
    pin = lambda a, bf=False: (torch.from_numpy(np.ascontiguousarray(a)).view(torch.bfloat16) if bf else torch.from_numpy(np.ascontiguousarray(a))).pin_memory()
    hq, hk, hv, hl, hd = pin(w.q_block, True), pin(w.k_new, True), pin(w.v_new, True), pin(aw.logits, True), pin(aw.drafts)
    h_out = torch.zeros((w.total_q, 32, 128), dtype=torch.bfloat16).pin_memory()
    h_acc, h_nxt, h_sl = (torch.full((60,), -7, dtype=torch.int32).pin_memory() for _ in range(3))
    ws = torch.empty(b.h.verify_step_host_workspace_bytes(w.prefix_len, w.q_len, "bf16", aw.logits.shape[1], aw.vocab), dtype=torch.uint8, device="cuda")
    b.h.verify_step_host(b.k_pool, b.v_pool, b.page_table, w.prefix_len, w.q_len, hq, hk, hv, hl, "bf16", aw.logits.shape[1], aw.vocab,
                         hd, h_out, h_acc, h_nxt, h_sl, ws)
    assert b.status() == 0
    kp, vp = oracle_pools_after_append(w)
    assert np.array_equal(host_storage(b.k_pool, "bf16"), kp) and np.array_equal(host_storage(b.v_pool, "bf16"), vp)
    ref, _ = oracle.attn_paged_batch(w.q_block, kp, vp, w.page_table, "bf16", w.prefix_len, w.q_len, w.cu_q)
    check_attention(h_out.to(torch.float64).numpy(), ref, "host step, 60 sequences")
    am, al, nt, sl = oracle.accept_greedy(aw.logits, "bf16", aw.vocab, aw.drafts, aw.cu_q, aw.prefix_len)
    assert np.array_equal(h_acc.numpy(), al) and np.array_equal(h_nxt.numpy(), nt) and np.array_equal(h_sl.numpy(), sl)


# ------------------------------------------------------------------ n-gram draft table (Sec. 4.3)
def _ngram_case(h, stream, n, contexts, k, fill):
    from oracle.toy_lm import build_ngram_table, ngram_drafts
    st = torch.tensor(stream, dtype=torch.int32, device="cuda")
    lut = torch.empty(agx.ngram_lut_bytes(len(stream)), dtype=torch.uint8, device="cuda")
    ws = torch.empty(agx.ngram_workspace_bytes(len(stream)), dtype=torch.uint8, device="cuda")
    h.ngram_build(st, n, lut, ws)
    B = len(contexts)
    ctx = torch.tensor(contexts, dtype=torch.int32, device="cuda").reshape(B, n - 1)
    fl = torch.tensor(fill, dtype=torch.int32, device="cuda").reshape(B, max(k, 1))[:, :k].contiguous()
    drafts = torch.full((B, max(k, 1)), -7, dtype=torch.int32, device="cuda")[:, :k].contiguous()
    has = torch.full((B,), -7, dtype=torch.int32, device="cuda")
    h.ngram_draft(lut, ctx, fl, k, drafts, has)
    torch.cuda.synchronize()
    table = build_ngram_table(stream, n)
    got_d, got_h = drafts.cpu().numpy(), has.cpu().numpy()
    for s in range(B):
        ref = ngram_drafts(table, contexts[s], k, n, fill=fill[s])
        if tuple(contexts[s]) not in table:
            assert ref is None and got_h[s] == 0     # selective fallback: no verify block for this sequence
        else:
            assert got_h[s] == 1 and got_d[s].tolist() == ref
    return table


@pytest.mark.parametrize("n", [2, 3])
def test_ngram_table_and_draft_chains_match_oracle(n):
    h = agx.Handle(32, 8, 128, "bf16")
    rng = np.random.default_rng(7 + n)
    ids = rng.choice(1 << 21, size=60, replace=False)            # a small alphabet of large ids: many repeats and count ties
    for length, alphabet in [(0, 4), (n - 1, 4), (n, 4), (37, 3), (1000, 12), (5000, 60), (120000, 60)]:
        stream = ids[rng.integers(0, alphabet, size=length)].tolist()
        k = 5
        known = [list(stream[i:i + n - 1]) for i in rng.integers(0, max(length - n + 1, 1), size=40)] if length >= n else []
        unknown = [[int(ids[59])] * (n - 1), [0] * (n - 1), [(1 << 21) - 1] * (n - 1), [-5] * (n - 1)]
        contexts = known + unknown
        fill = ids[rng.integers(0, alphabet, size=(len(contexts), k))].tolist()
        table = _ngram_case(h, stream, n, contexts, k, fill)
        if length >= 1000:   # every key of the table, one lookup each
            keys = [list(key) for key in table]
            _ngram_case(h, stream, n, keys, 1, [[0]] * len(keys))
    assert h.get_status() == 0


def test_ngram_build_flags_tokens_outside_its_range_and_skips_their_windows():
    h = agx.Handle(32, 8, 128, "bf16")
    stream = [5, 6, 7, 1 << 21, 5, 6, 9, -1, 5, 6, 9]
    from oracle.toy_lm import build_ngram_table
    st = torch.tensor(stream, dtype=torch.int32, device="cuda")
    lut = torch.empty(agx.ngram_lut_bytes(len(stream)), dtype=torch.uint8, device="cuda")
    ws = torch.empty(agx.ngram_workspace_bytes(len(stream)), dtype=torch.uint8, device="cuda")
    h.ngram_build(st, 3, lut, ws)
    ctx = torch.tensor([[5, 6], [6, 7]], dtype=torch.int32, device="cuda")
    fl = torch.zeros((2, 1), dtype=torch.int32, device="cuda")
    d = torch.zeros((2, 1), dtype=torch.int32, device="cuda"); hs = torch.zeros(2, dtype=torch.int32, device="cuda")
    h.ngram_draft(lut, ctx, fl, 1, d, hs)
    torch.cuda.synchronize()
    assert h.get_status() & agx.AGX_DEV_BAD_TOKEN
    assert d[0, 0].item() == 9 and hs.tolist() == [1, 0]     # (5,6)->9 twice, ->7 once; (6,7,bad) skipped
    with pytest.raises(agx.AgxError):
        h.ngram_build(st, 4, lut, ws)


def test_speculative_loop_on_gpu_emits_the_tokens_of_plain_greedy_decoding():
    """Greedy speculative decoding (verify blocks through agx_kv_append / agx_attn_prefixed / agx_accept_greedy,
    drafts from the device-side trigram table with its selective fallback) emits exactly the stream of
    one-token-at-a-time greedy decoding, on the GPU and in the oracle (Sec. 2.3, Sec. 4.3)."""
    from oracle.toy_lm import ToyLM
    from tests.spec_loop import CudaBackend, DeviceNgramDrafts, OracleBackend, generate
    lm = ToyLM(seed=11)
    rng = np.random.default_rng(21)
    motif = rng.integers(0, lm.vocab, size=12).tolist()
    prompt = (motif * 4)[:40]
    T = 48
    base, calls0, _ = generate(OracleBackend(lm), prompt, T)
    plain, calls1, _ = generate(CudaBackend(lm), prompt, T)
    spec, calls2, acc = generate(CudaBackend(lm), prompt, T, DeviceNgramDrafts(prompt, 3, vocab=lm.vocab), k=4)
    wrong, calls3, acc_w = generate(CudaBackend(lm), prompt, T, lambda hist, k: [(hist[-1] + 1 + i) % lm.vocab for i in range(k)], k=4)
    assert plain == base and spec == base and wrong == base
    assert calls1 == T and calls2 <= T and calls3 <= T


# ------------------------------------------------------------------ argument errors (host side)
def test_argument_errors_are_reported_not_faulted():
    w = W.make_attn_workload("err", 6, "bf16", 32, 8, 128, [100], [4])
    b = DeviceBatch(w)
    with pytest.raises(agx.AgxError) as e:
        b.h.attn_prefixed(b.q_block, b.k_pool, b.v_pool, b.page_table, [100], [0], b.out)
    assert e.value.status == -1
    with pytest.raises(agx.AgxError) as e:
        b.h.attn_prefixed(b.q_block, b.k_pool, b.v_pool, b.page_table, [100000], [4], b.out)
    assert e.value.status == -2
    with pytest.raises(agx.AgxError):
        agx.Handle(32, 5, 128, "bf16")
    with pytest.raises(agx.AgxError):
        agx.Handle(32, 8, 96, "bf16")
    w2 = W.c2_decode_verify()
    b2 = DeviceBatch(w2)
    with pytest.raises(agx.AgxError) as e:  # split launch without workspace
        b2.h.attn_prefixed(b2.q_block, b2.k_pool, b2.v_pool, b2.page_table, w2.prefix_len, w2.q_len, b2.out)
    assert e.value.status == -1


# ------------------------------------------------------------------ tensor-core stream schedule (few rows, long context)
@pytest.mark.parametrize("P,q,hq,hkv", [
    (0, 1, 32, 8), (1, 1, 32, 8), (15, 1, 8, 8), (17, 4, 32, 8), (127, 8, 32, 8), (128, 8, 32, 8), (129, 16, 32, 8),
    (255, 2, 32, 8), (1000, 3, 24, 8), (2049, 5, 32, 8), (5000, 8, 32, 8), (777, 32, 32, 8), (300, 7, 4, 1),
    (130, 100, 4, 4), (4095, 2, 16, 2), (20000, 8, 32, 8), (9000, 25, 32, 8),
])
def test_stream_schedule_shapes(P, q, hq, hkv, monkeypatch):
    """Blocks of at most 128 query rows per KV head on the tcgen05 kernel whose two softmax warpgroups
    alternate KV tiles; forced here for every context length."""
    monkeypatch.setenv("AGX_STREAM_MIN_TOKENS", "0")
    w = W.make_attn_workload(f"stream_{P}_{q}", 3000 + P + q, "bf16", hq, hkv, 128, [P], [q], spare_pages=3)
    run_and_check(w, sample=(13, 64) if P > 6000 else None, poison=True)


@pytest.mark.parametrize("P,q,hq,hkv", [
    (700, 80, 32, 8),      # 320 rows per KV head: three 128-row chunks, the last half empty
    (100, 90, 6, 2),       # G = 3, 270 rows, prefix not page-aligned
    (1500, 33, 32, 8),     # 132 rows: a second chunk of 4 rows
    (0, 96, 16, 4),        # pure causal block of 384 rows: chunks that see nothing of the later KV splits
])
def test_stream_schedule_with_several_row_chunks(P, q, hq, hkv):
    """Blocks of 129..384 rows per KV head take the one-Q-tile schedule in 128-row chunks (short suffixes over short
    prefixes, where its lower fixed costs beat the 256-row schedule): every output row against the oracle, in the
    two-call and in the fused form."""
    w = W.make_attn_workload(f"chunks_{P}_{q}", 3000 + P + q, "bf16", hq, hkv, 128, [P], [q], spare_pages=2)
    run_and_check(w, poison=True)
    run_and_check(w, poison=True, fused=True)


def test_stream_schedule_ragged_batch_matches_warp_mma_kernel(monkeypatch):
    P = [2048, 2100, 4000, 2048 + 15, 9000, 2500, 3001, 2048]
    q = [1, 2, 4, 8, 16, 3, 5, 30]
    w = W.make_attn_workload("ragged_stream", 43, "bf16", 32, 8, 128, P, q, shared_prefix_tokens=2048)
    monkeypatch.setenv("AGX_STREAM_MIN_TOKENS", "0")
    b = DeviceBatch(w); b.append(); a, _ = b.attend()
    monkeypatch.setenv("AGX_STREAM_MIN_TOKENS", "100000000")
    b2 = DeviceBatch(w); b2.append(); c, _ = b2.attend()
    assert b.status() == 0 and b2.status() == 0
    assert np.max(np.abs(a - c)) < 2e-2
    run_and_check(w, sample=(7, 12))


# ------------------------------------------------------------------ append fused into the attention launch
FUSED_CASES = [
    # name, dtype, hq, hkv, d, P, q, stream schedule forced
    ("decode", "bf16", 32, 8, 128, [0, 1, 15, 16, 4095], [1, 1, 1, 1, 1], False),
    ("verify_ragged", "bf16", 32, 8, 128, [2048, 2100, 4000, 2063, 9000, 2500, 3001, 250], [1, 2, 4, 8, 16, 3, 5, 30], False),
    ("verify_split_boundaries", "bf16", 32, 8, 128, [249, 255, 256, 511, 1020], [8, 8, 8, 8, 8], False),
    ("stream_forced", "bf16", 32, 8, 128, [17, 127, 2049, 5000, 777], [4, 8, 5, 8, 32], True),
    ("stream_long", "bf16", 32, 8, 128, [20000, 14000], [8, 3], False),
    ("mid_q", "bf16", 32, 8, 128, [3000, 130], [20, 9], False),
    ("tile_one_chunk", "bf16", 8, 2, 128, [256, 100, 1000], [64, 50, 33], False),
    ("tile_many_chunks", "bf16", 24, 8, 128, [1030, 5], [300, 200], False),
    ("mixed_kinds", "bf16", 32, 8, 128, [2048, 2300, 2055, 4000, 2600, 3000], [8, 200, 1, 130, 16, 513], False),
    ("fp32", "f32", 8, 2, 64, [256, 30, 0], [4, 1, 7], False),
]


@pytest.mark.parametrize("name,dtype,hq,hkv,d,P,q,stream", FUSED_CASES, ids=[c[0] for c in FUSED_CASES])
def test_fused_append_attention_equals_the_two_calls_and_the_oracle(name, dtype, hq, hkv, d, P, q, stream, monkeypatch):
    """agx_attn_prefixed_append: pools and outputs bit-identical to agx_kv_append followed by agx_attn_prefixed
    (the same kernels do the arithmetic), slots it must not touch unchanged, and parity with the oracle."""
    if stream:
        monkeypatch.setenv("AGX_STREAM_MIN_TOKENS", "0")
    w = W.make_attn_workload("fused_" + name, 7000 + sum(P) + sum(q), dtype, hq, hkv, d, P, q, spare_pages=3)
    two = DeviceBatch(w); two.append(); out2, lse2 = two.attend()
    one = DeviceBatch(w); out1, lse1 = one.attend_append()
    assert one.status() == 0 and two.status() == 0
    assert torch.equal(one.k_pool, two.k_pool) and torch.equal(one.v_pool, two.v_pool)
    assert np.array_equal(out1, out2) and np.array_equal(lse1, lse2)
    run_and_check(w, sample=(3, 40) if max(P) + max(q) > 3000 else None, fused=True)


def test_fused_append_saves_the_append_launch_on_a_verify_batch():
    w = W.c2_decode_verify()
    b = DeviceBatch(w); b.attend_append()
    fused = b.launches
    b2 = DeviceBatch(w); b2.append(); b2.attend()
    assert fused == b2.launches and b.status() == 0      # attention + combine; the append took a launch of its own before
    assert torch.equal(b.k_pool, b2.k_pool) and torch.equal(b.out, b2.out)


def test_fused_append_reports_a_bad_page_and_skips_the_row():
    w = W.make_attn_workload("fused_bad_page", 77, "bf16", 32, 8, 128, [40, 300], [8, 8], spare_pages=2)
    b = DeviceBatch(w)
    pt = w.page_table.copy(); pt[1, 300 // 16] = w.k_pool.shape[0] + 5
    b.page_table = dev(pt)
    before = b.k_pool.clone()
    b.attend_append()
    assert b.status() & agx.AGX_DEV_BAD_PAGE
    touched = (b.k_pool != before).flatten(1).any(1).nonzero().flatten().cpu().numpy()
    assert int(w.page_table[1, 300 // 16]) not in touched.tolist()      # the row behind the bad id was not written anywhere
    assert set(touched.tolist()) == {int(w.page_table[0, 2]), int(w.page_table[1, 19])}


# ------------------------------------------------------------------ tensor-core tile kernel (large q)
@pytest.mark.parametrize("P,q,hq,hkv", [
    (0, 128, 8, 2),        # pure causal prefill, G = 4, one tile pair, exact multiples
    (256, 64, 8, 2),       # 256 rows: exactly one CTA chunk
    (100, 90, 6, 2),       # G = 3, ragged rows, P not page-aligned
    (777, 130, 32, 8),     # L % 16 != 0 (ragged last page), several chunks
    (3000, 40, 32, 8),     # 160 rows: tile B mostly padding
    (1030, 300, 24, 8),    # G = 3, several KV splits
    (5, 200, 4, 4),        # G = 1 (MHA)
])
def test_tile_kernel_shapes(P, q, hq, hkv):
    w = W.make_attn_workload(f"tile_{P}_{q}", 2000 + P + q, "bf16", hq, hkv, 128, [P], [q], spare_pages=2)
    run_and_check(w, poison=True)   # every output row


def test_c3_prefix_cached_prefill_and_full_prefill_rows():
    """Prefix-cached prefill (P = 3072, q = 512, 24/8 heads) against the oracle, and the oracle's own
    check that these rows equal rows 3072.. of a full 3584-token uncached prefill."""
    w = W.c3_prefix_prefill()
    b, stats = run_and_check(w, strict=True)   # every output row
    out = b.out.to(torch.float64).cpu().numpy()
    kp, vp = oracle_pools_after_append(w)
    P, q = 3072, 512
    K = W.gather_contiguous(kp, w.page_table[0], P + q); V = W.gather_contiguous(vp, w.page_table[0], P + q)
    rng = np.random.default_rng(1)
    si = rng.integers(0, q, 40).astype(np.int32); sh = rng.integers(0, 24, 40).astype(np.int32)
    Qfull = np.zeros((P + q, 24, 128), dtype=np.uint16); Qfull[P:] = w.q_block
    full, _, _ = oracle.attn_contiguous(Qfull, K, V, "bf16", 0, select=(si + P, sh))
    check_attention(out[si, sh], full, "c3 vs full prefill rows", strict=True)


def test_order_of_sequences_inside_a_launch_changes_no_bit(monkeypatch):
    """The planner puts the longest contexts first in the launches of the tensor-core schedules; with
    AGX_LONGEST_FIRST=0 they stay in batch order.  Work items do not depend on one another, so the two orders must
    give the same bits (ragged prefill blocks and verify blocks in one batch, shortest context first in the batch)."""
    w = W.make_attn_workload("order", 4242, "bf16", 32, 8, 128, [300, 9000, 1500, 12000, 4000, 700], [200, 8, 500, 4, 300, 130],
                             spare_pages=2)
    outs = []
    for flag in ("1", "0"):
        monkeypatch.setenv("AGX_LONGEST_FIRST", flag)
        b = DeviceBatch(w)
        out, lse = b.attend_append()
        assert b.status() == 0
        outs.append((host_storage(b.out, "bf16").copy(), lse.copy()))
    assert np.array_equal(outs[0][0], outs[1][0]) and np.array_equal(outs[0][1], outs[1][1])
    kp, vp = oracle_pools_after_append(w)
    rng = np.random.default_rng(7)
    for s in range(w.batch):
        q = int(w.q_len[s]); r0 = int(w.cu_q[s])
        si = rng.integers(0, q, 8).astype(np.int32); sh = rng.integers(0, 32, 8).astype(np.int32)
        ref, _, _ = oracle.attn_paged(w.q_block[r0:r0 + q], kp, vp, w.page_table[s], "bf16", int(w.prefix_len[s]), select=(si, sh))
        got = torch.from_numpy(outs[0][0].view(np.int16)).view(torch.bfloat16).to(torch.float64).numpy()
        check_attention(got[r0 + si, sh], ref, "order of sequences")


def test_tile_and_small_kernels_in_one_ragged_batch():
    P = [2048, 2300, 2048 + 7, 4000, 2600, 3000]
    q = [8, 200, 1, 130, 16, 513]
    w = W.make_attn_workload("mixed", 91, "bf16", 32, 8, 128, P, q, shared_prefix_tokens=2048)
    b, _ = run_and_check(w)   # every output row
    assert b.launches >= 3


def test_tile_kernel_matches_mma_sync_baseline(monkeypatch):
    w = W.make_attn_workload("tile_vs_mma", 17, "bf16", 32, 8, 128, [900], [260])
    b = DeviceBatch(w); b.append(); a, _ = b.attend()
    monkeypatch.setenv("AGX_FORCE_MMA_SYNC", "1")
    b2 = DeviceBatch(w); b2.append(); c, _ = b2.attend()
    assert np.max(np.abs(a - c)) < 2e-2


# ------------------------------------------------------------------ handle options
@pytest.mark.parametrize("name,hq,hkv,P,q,env", [
    ("warp-mma", 32, 8, [4096], [8], {}),
    ("warp-mma batch", 32, 8, [700, 45, 2000, 16], [8, 3, 1, 16], {}),
    ("stream", 32, 8, [9000, 8200], [8, 16], {}),
    ("tile", 24, 8, [3072], [512], {}),
    ("tile, prefix not page-aligned", 32, 8, [1003, 130], [200, 77], {}),
])
def test_early_prefix_loads_change_nothing(name, hq, hkv, P, q, env, monkeypatch):
    """AGX_OPT_EARLY_PREFIX_LOADS only moves loads of cached-prefix pages in front of the dependency wait: with the
    option on, a chain of (append, attention) pairs whose block rows change every round must give, bit for bit,
    what the same chain gives with the option off - in the two-call form, where the rows read were written by
    the launch directly in front, and in the fused form."""
    w = W.make_attn_workload("early_" + name, 77, "bf16", hq, hkv, 128, P, q)
    outs = {}
    for early in (0, 1):
        b = DeviceBatch(w)
        b.h.set_option(agx.AGX_OPT_EARLY_PREFIX_LOADS, early)
        g = torch.Generator(device="cuda"); g.manual_seed(5)
        got = []
        for it in range(6):
            b.k_new.copy_(torch.randn(b.k_new.shape, generator=g, device="cuda").to(torch.bfloat16))
            b.v_new.copy_(torch.randn(b.v_new.shape, generator=g, device="cuda").to(torch.bfloat16))
            if it % 2 == 0:
                b.append()
                b.h.attn_prefixed(b.q_block, b.k_pool, b.v_pool, b.page_table, w.prefix_len, w.q_len, b.out, b.lse, b.ws)
            else:
                b.h.attn_prefixed_append(b.q_block, b.k_new, b.v_new, b.k_pool, b.v_pool, b.page_table, w.prefix_len,
                                         w.q_len, b.out, b.lse, b.ws)
            got.append(b.out.clone())
        torch.cuda.synchronize()
        assert b.status() == 0
        outs[early] = got
    for a, c in zip(outs[0], outs[1]):
        assert torch.equal(a, c)
    # and the last round against the oracle
    w.k_new[:] = host_storage(b.k_new, "bf16"); w.v_new[:] = host_storage(b.v_new, "bf16")
    kp, vp = oracle_pools_after_append(w)
    ref, _ = oracle.attn_paged_batch(w.q_block, kp, vp, w.page_table, w.dtype, w.prefix_len, w.q_len, w.cu_q)
    check_attention(outs[1][-1].to(torch.float64).cpu().numpy(), ref, name)


@pytest.mark.parametrize("name,hq,hkv,P,q,stage,env", [
    ("warp-mma kernel", 4, 1, [300], [8], 0, {}),
    ("warp-mma kernel, later stage", 4, 1, [900], [4], 2, {"AGX_SMALL_MIN_SPLIT": "1024"}),      # one CTA per KV head, 8 stages
    ("stream schedule", 4, 1, [500], [20], 0, {}),
    ("stream schedule, later tile", 4, 1, [900], [20], 3, {"AGX_TILE_SPLIT_TOKENS": "1024"}),   # one split of 8 tiles
    ("256-row schedule", 4, 1, [300], [100], 0, {}),
    ("256-row schedule, later tile", 4, 1, [700], [100], 2, {"AGX_TILE_SPLIT_TOKENS": "1024"}),
])
def test_a_wait_that_runs_out_sets_the_status_and_leaves_the_handle_usable(name, hq, hkv, P, q, stage, env, monkeypatch):
    """The give-up path of the bounded in-kernel waits.  With the wait limit cut to 2e5 clock ticks and the test
    hook that makes the copy-issuing warp leave one K/V stage out (nothing is armed, nothing is copied - a flag that
    nothing sets), the consumers' waits for that stage run out: the call returns, the device status carries
    AGX_DEV_WAIT_TIMEOUT, and the next ordinary call on the same handle gives bit for bit what a fresh handle gives."""
    for k, v in env.items():
        monkeypatch.setenv(k, v)
    w = W.make_attn_workload("timeout_" + name, 88, "bf16", hq, hkv, 128, P, q)
    fresh = DeviceBatch(w); fresh.append(); fresh.attend()
    assert fresh.status() == 0
    b = DeviceBatch(w); b.append()
    b.h.set_option(agx.AGX_OPT_WAIT_LIMIT_CYCLES, 200000)
    b.h.set_option(agx.AGX_OPT_TEST_DROP_STAGE, stage)
    b.attend()                                   # returns (synchronises) although a stage never arrived
    assert b.status() & agx.AGX_DEV_WAIT_TIMEOUT
    assert b.status() == 0                       # reading the status cleared it
    b.h.set_option(agx.AGX_OPT_TEST_DROP_STAGE, -1)
    b.h.set_option(agx.AGX_OPT_WAIT_LIMIT_CYCLES, 4000000000)
    b.out.zero_()
    b.attend()
    assert b.status() == 0
    assert torch.equal(b.out, fresh.out) and torch.equal(b.lse, fresh.lse)


def test_set_option_rejects_what_it_does_not_know():
    h = agx.Handle(32, 8, 128, "bf16")
    with pytest.raises(agx.AgxError) as e:
        h.set_option(99, 1)
    assert e.value.status == -1
    with pytest.raises(agx.AgxError) as e:
        h.set_option(agx.AGX_OPT_WAIT_LIMIT_CYCLES, 10)
    assert e.value.status == -2
