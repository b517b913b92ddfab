"""Pins for the CPU oracle: closed forms, invariants, library routines, brute force and the
paper's structural worked example.  None of these compares the oracle with itself through the
same formula; each is chosen so a plausible slip (wrong causal bound, wrong GQA map, dropped
scale, transposed page index, tie rule) fails at least one."""
import math
import os

import numpy as np
import pytest

import oracle
from paper_2605_10380_b200 import workloads as W

GOLDEN = os.path.join(os.path.dirname(__file__), "golden")


def _rand(rng, shape, dtype="f32"):
    return W.to_storage(rng.standard_normal(shape, dtype=np.float32), dtype)


def _small(seed=0, P=37, q=5, hq=4, hkv=2, d=8, dtype="f32"):
    rng = np.random.default_rng(seed)
    L = P + q
    return (_rand(rng, (q, hq, d), dtype), _rand(rng, (L, hkv, d), dtype), _rand(rng, (L, hkv, d), dtype))


# ------------------------------------------------------------------ brute force (pure Python floats)
def brute_attention(Q, K, V, P, scale):
    q, hq, d = Q.shape
    hkv = K.shape[1]
    G = hq // hkv
    out = [[[0.0] * d for _ in range(hq)] for _ in range(q)]
    for i in range(q):
        for h in range(hq):
            g = h // G
            scores = []
            for j in range(P + i + 1):
                acc = 0.0
                for c in range(d):
                    acc += float(Q[i, h, c]) * float(K[j, g, c])
                scores.append(acc * scale)
            top = max(scores)
            ws = [math.exp(s - top) for s in scores]
            z = math.fsum(ws)
            for c in range(d):
                out[i][h][c] = math.fsum(w * float(V[j, g, c]) for j, w in enumerate(ws)) / z
    return np.array(out)


@pytest.mark.parametrize("P,q", [(0, 1), (0, 7), (1, 1), (15, 1), (16, 3), (17, 7), (5, 19), (23, 1)])
def test_brute_force_tiny(P, q):
    Q, K, V = _small(seed=P * 31 + q, P=P, q=q, hq=4, hkv=2, d=8)
    scale = 0.37
    out, lse, ps = oracle.attn_contiguous(Q, K, V, "f32", P, scale=scale)
    ref = brute_attention(Q, K, V, P, scale)
    np.testing.assert_allclose(out, ref, rtol=0, atol=1e-13)


def test_brute_force_bf16_storage():
    Q, K, V = _small(seed=3, P=9, q=4, hq=6, hkv=2, d=8, dtype="bf16")
    out, _, _ = oracle.attn_contiguous(Q, K, V, "bf16", 9)
    Qf, Kf, Vf = (W.bf16_bits_to_f32(a) for a in (Q, K, V))
    ref = brute_attention(Qf, Kf, Vf, 9, 1.0 / math.sqrt(8))
    np.testing.assert_allclose(out, ref, rtol=0, atol=1e-13)


# ------------------------------------------------------------------ library routine
@pytest.mark.parametrize("P,q,hq,hkv,d", [(40, 9, 8, 2, 16), (0, 12, 4, 4, 32), (129, 1, 6, 3, 64)])
def test_against_torch_sdpa_fp64(P, q, hq, hkv, d):
    import torch
    Q, K, V = _small(seed=7, P=P, q=q, hq=hq, hkv=hkv, d=d)
    out, lse, _ = oracle.attn_contiguous(Q, K, V, "f32", P)
    L = P + q
    G = hq // hkv
    tq = torch.from_numpy(Q.astype(np.float64)).permute(1, 0, 2)  # [hq, q, d]
    tk = torch.from_numpy(K.astype(np.float64)).permute(1, 0, 2).repeat_interleave(G, dim=0)
    tv = torch.from_numpy(V.astype(np.float64)).permute(1, 0, 2).repeat_interleave(G, dim=0)
    mask = torch.arange(L)[None, :] <= (P + torch.arange(q))[:, None]
    ref = torch.nn.functional.scaled_dot_product_attention(tq, tk, tv, attn_mask=mask)
    np.testing.assert_allclose(out, ref.permute(1, 0, 2).numpy(), rtol=0, atol=1e-12)
    logits = torch.einsum("hqd,hkd->hqk", tq, tk) / math.sqrt(d)
    ref_lse = torch.logsumexp(logits.masked_fill(~mask, -float("inf")), dim=-1)
    np.testing.assert_allclose(lse, ref_lse.T.numpy(), rtol=0, atol=1e-12)


# ------------------------------------------------------------------ the five required self-checks
def test_check1_rows_sum_to_one():
    Q, K, V = _small(seed=1, P=300, q=6, hq=8, hkv=2, d=16)
    _, _, ps = oracle.attn_contiguous(Q, K, V, "f32", 300)
    assert np.max(np.abs(ps - 1.0)) < 1e-12


def test_check2_q1_is_plain_decode():
    for dtype in ("f32", "bf16"):
        Q, K, V = _small(seed=2, P=211, q=1, hq=8, hkv=4, d=32, dtype=dtype)
        out, _, _ = oracle.attn_contiguous(Q, K, V, dtype, 211)
        ref = oracle.decode_plain(Q[0], K, V, dtype)
        np.testing.assert_allclose(out[0], ref, rtol=0, atol=1e-13)


def _paged_copy(rng, K, V, spare=5):
    L, hkv, d = K.shape
    npg = W.pages_needed(L)
    perm = rng.permutation(npg + spare).astype(np.int32)
    row = perm[:npg]
    kp = _rand(rng, (npg + spare, hkv, 16, d), "f32" if K.dtype == np.float32 else "bf16")
    vp = _rand(rng, (npg + spare, hkv, 16, d), "f32" if K.dtype == np.float32 else "bf16")
    W.scatter_contiguous(kp, row, 0, K)
    W.scatter_contiguous(vp, row, 0, V)
    return kp, vp, row


@pytest.mark.parametrize("dtype", ["f32", "bf16"])
def test_check3_paged_equals_contiguous_bitwise(dtype):
    rng = np.random.default_rng(33)
    Q, K, V = _small(seed=4, P=100, q=7, hq=4, hkv=2, d=16, dtype=dtype)
    kp, vp, row = _paged_copy(rng, K, V)
    a, la, _ = oracle.attn_contiguous(Q, K, V, dtype, 100)
    b, lb, _ = oracle.attn_paged(Q, kp, vp, row, dtype, 100)
    assert np.array_equal(a, b) and np.array_equal(la, lb)
    # and the gather helper returns what was scattered
    assert np.array_equal(W.gather_contiguous(kp, row, 107), K)


def test_check4_prefix_cached_equals_rows_of_full_prefill():
    """Sec. 2.3 prefix caching is exact: computing only the uncached suffix over the cached
    prefix gives the same rows as prefilling the whole prompt from scratch."""
    rng = np.random.default_rng(44)
    P, q, hq, hkv, d = 75, 21, 6, 2, 16
    L = P + q
    Qfull = _rand(rng, (L, hq, d)); K = _rand(rng, (L, hkv, d)); V = _rand(rng, (L, hkv, d))
    full, lse_full, _ = oracle.attn_contiguous(Qfull, K, V, "f32", 0)  # P=0, q=L: uncached prefill
    kp, vp, row = _paged_copy(rng, K, V)
    part, lse_part, _ = oracle.attn_paged(Qfull[P:], kp, vp, row, "f32", P)
    np.testing.assert_allclose(part, full[P:], rtol=0, atol=1e-12)
    np.testing.assert_allclose(lse_part, lse_full[P:], rtol=0, atol=1e-12)


def test_check4_config3_shape_sampled():
    """Same claim at the prefix-cached prefill configuration's real size (3072 + 512, 24/8 heads,
    d=128, bf16), on sampled rows so the CPU suite stays short."""
    w = W.c3_prefix_prefill()
    P, q = int(w.prefix_len[0]), int(w.q_len[0])
    kp, vp = w.k_pool.copy(), w.v_pool.copy()
    oracle.kv_append(kp, vp, w.k_new, w.v_new, "bf16", w.page_table, w.prefix_len, w.cu_q)
    K = W.gather_contiguous(kp, w.page_table[0], P + q)
    V = W.gather_contiguous(vp, w.page_table[0], P + q)
    rng = np.random.default_rng(0)
    si = np.concatenate([[0, q - 1], rng.integers(0, q, 30)]).astype(np.int32)
    sh = np.concatenate([[0, 23], rng.integers(0, 24, 30)]).astype(np.int32)
    part, _, ps = oracle.attn_paged(w.q_block, kp, vp, w.page_table[0], "bf16", P, select=(si, sh))
    # full uncached prefill of all 3584 tokens: its query rows 0..3071 are irrelevant to the
    # sampled outputs, so only the sampled rows of the P=0 problem are evaluated.
    Qfull = np.zeros((P + q, 24, 128), dtype=np.uint16)
    Qfull[P:] = w.q_block
    full, _, _ = oracle.attn_contiguous(Qfull, K, V, "bf16", 0, select=(si + P, sh))
    np.testing.assert_allclose(part, full, rtol=0, atol=1e-12)
    assert np.max(np.abs(ps - 1)) < 1e-12


# ------------------------------------------------------------------ closed forms
def test_closed_form_equal_value_rows():
    Q, K, V = _small(seed=5, P=50, q=3)
    V[:] = V[0:1]
    out, _, _ = oracle.attn_contiguous(Q, K, V, "f32", 50)
    G = 2
    for h in range(4):
        np.testing.assert_allclose(out[:, h, :], np.broadcast_to(V[0, h // G].astype(np.float64), (3, 8)), atol=1e-14)


def test_closed_form_zero_query_is_running_mean_and_pins_causal_boundary():
    P, q, hq, hkv, d = 29, 6, 2, 1, 4
    rng = np.random.default_rng(6)
    Q = np.zeros((q, hq, d), dtype=np.float32)
    K = _rand(rng, (P + q, hkv, d))
    V = np.zeros((P + q, hkv, d), dtype=np.float32)
    V[:, 0, :] = np.arange(P + q, dtype=np.float32)[:, None]  # ramp V[j] = j
    out, lse, _ = oracle.attn_contiguous(Q, K, V, "f32", P)
    for i in range(q):
        np.testing.assert_allclose(out[i], (P + i) / 2.0, atol=1e-12)  # mean of 0..P+i
        np.testing.assert_allclose(lse[i], math.log(P + i + 1), atol=1e-13)


def test_closed_form_equal_key_rows_give_uniform_weights():
    Q, K, V = _small(seed=8, P=20, q=2)
    K[:] = K[0:1]
    out, _, _ = oracle.attn_contiguous(Q, K, V, "f32", 20)
    for i in range(2):
        for h in range(4):
            np.testing.assert_allclose(out[i, h], V[: 20 + i + 1, h // 2].astype(np.float64).mean(0), atol=1e-13)


def test_closed_form_dominant_key_and_scale():
    P, q, d = 30, 1, 8
    Q = np.zeros((1, 1, d), dtype=np.float32); Q[0, 0, 0] = 1.0
    K = np.zeros((P + 1, 1, d), dtype=np.float32); K[17, 0, 0] = 200.0
    rng = np.random.default_rng(9)
    V = _rand(rng, (P + 1, 1, d))
    out, _, _ = oracle.attn_contiguous(Q, K, V, "f32", P, scale=0.5)  # score gap = 100
    np.testing.assert_allclose(out[0, 0], V[17, 0].astype(np.float64), atol=1e-30 + 31 * math.exp(-100) * 10)
    # scale really multiplies the score: two keys, gap g -> weights sigmoid(scale*g)
    K2 = np.zeros((2, 1, d), dtype=np.float32); K2[1, 0, 0] = 3.0
    V2 = np.zeros((2, 1, d), dtype=np.float32); V2[1, 0, :] = 1.0
    o2, _, _ = oracle.attn_contiguous(Q, K2, V2, "f32", 1, scale=0.25)
    np.testing.assert_allclose(o2[0, 0], 1.0 / (1.0 + math.exp(-0.75)), atol=1e-15)
    # default scale is 1/sqrt(d)
    o3, _, _ = oracle.attn_contiguous(Q, K2, V2, "f32", 1)
    np.testing.assert_allclose(o3[0, 0], 1.0 / (1.0 + math.exp(-3.0 / math.sqrt(d))), atol=1e-15)


# ------------------------------------------------------------------ invariants
def test_invariant_prefix_permutation():
    Q, K, V = _small(seed=10, P=64, q=4)
    rng = np.random.default_rng(1)
    perm = np.concatenate([rng.permutation(64), np.arange(64, 68)])
    a, _, _ = oracle.attn_contiguous(Q, K, V, "f32", 64)
    b, _, _ = oracle.attn_contiguous(Q, K[perm], V[perm], "f32", 64)
    np.testing.assert_allclose(a, b, atol=1e-13)
    # permuting the in-block rows is NOT an invariance (causal order matters)
    perm2 = np.concatenate([np.arange(64), [67, 66, 65, 64]])
    c, _, _ = oracle.attn_contiguous(Q, K[perm2], V[perm2], "f32", 64)
    assert np.max(np.abs(a - c)) > 1e-3


def test_invariant_gqa_equals_mha_with_replicated_heads():
    Q, K, V = _small(seed=11, P=33, q=3, hq=6, hkv=2, d=8)
    a, _, _ = oracle.attn_contiguous(Q, K, V, "f32", 33)
    Kr, Vr = np.repeat(K, 3, axis=1), np.repeat(V, 3, axis=1)
    b, _, _ = oracle.attn_contiguous(Q, Kr, Vr, "f32", 33)
    np.testing.assert_allclose(a, b, atol=1e-14)
    # heads 0..2 use kv head 0, heads 3..5 kv head 1 (contiguous groups)
    Kx = K.copy(); Kx[:, 1] *= -1.0
    c, _, _ = oracle.attn_contiguous(Q, Kx, V, "f32", 33)
    assert np.array_equal(a[:, :3], c[:, :3]) and not np.allclose(a[:, 3:], c[:, 3:])


def test_invariant_split_and_merge():
    """(m, l, O) partials over any partition of the keys merge to the unsplit result."""
    P, q = 90, 1
    Q, K, V = _small(seed=12, P=P, q=q, hq=2, hkv=1, d=8)
    full, lse, _ = oracle.attn_contiguous(Q, K, V, "f32", P)
    cuts = [0, 13, 48, 49, 91]
    parts = []
    for a, b in zip(cuts[:-1], cuts[1:]):
        o, l, _ = oracle.attn_contiguous(Q, K[a:b], V[a:b], "f32", b - a - 1)
        parts.append((o, l))
    m = np.max([l for _, l in parts], axis=0)
    wsum = sum(np.exp(l - m) for _, l in parts)
    merged = sum(o * np.exp(l - m)[..., None] for o, l in parts) / wsum[..., None]
    np.testing.assert_allclose(merged, full, atol=1e-13)
    np.testing.assert_allclose(m + np.log(wsum), lse, atol=1e-13)


def test_invariant_slots_beyond_length_are_ignored():
    rng = np.random.default_rng(13)
    Q, K, V = _small(seed=13, P=21, q=2, hq=2, hkv=1, d=8)
    kp, vp, row = _paged_copy(rng, K, V)
    a, _, _ = oracle.attn_paged(Q, kp, vp, row, "f32", 21)
    kp2, vp2 = kp.copy(), vp.copy()
    kp2[row[1], :, 7:, :] = np.nan  # tokens 23.. of page 1 are beyond P+q = 23
    vp2[row[1], :, 7:, :] = np.nan
    b, _, _ = oracle.attn_paged(Q, kp2, vp2, row, "f32", 21)
    assert np.array_equal(a, b)


def test_kv_append_places_rows_and_touches_nothing_else():
    w = W.make_attn_workload("t", 77, "bf16", 4, 2, 8, [5, 30, 16], [3, 1, 20], spare_pages=3)
    kp, vp = w.k_pool.copy(), w.v_pool.copy()
    oracle.kv_append(kp, vp, w.k_new, w.v_new, "bf16", w.page_table, w.prefix_len, w.cu_q)
    touched = np.zeros(kp.shape[:3] + (1,), dtype=bool)
    for s in range(3):
        for r in range(int(w.cu_q[s]), int(w.cu_q[s + 1])):
            tok = int(w.prefix_len[s]) + r - int(w.cu_q[s])
            pg = int(w.page_table[s, tok // 16])
            assert np.array_equal(kp[pg, :, tok % 16, :], w.k_new[r])
            assert np.array_equal(vp[pg, :, tok % 16, :], w.v_new[r])
            touched[pg, :, tok % 16] = True
    keep = ~np.broadcast_to(touched, kp.shape)
    assert np.array_equal(kp[keep], w.k_pool[keep]) and np.array_equal(vp[keep], w.v_pool[keep])


def test_batch_form_matches_per_sequence_calls():
    w = W.make_attn_workload("t", 78, "f32", 4, 2, 8, [5, 30, 16], [3, 1, 20], shared_prefix_tokens=0)
    kp, vp = w.k_pool.copy(), w.v_pool.copy()
    oracle.kv_append(kp, vp, w.k_new, w.v_new, "f32", w.page_table, w.prefix_len, w.cu_q)
    out, lse = oracle.attn_paged_batch(w.q_block, kp, vp, w.page_table, "f32", w.prefix_len, w.q_len, w.cu_q)
    for s in range(3):
        a, b = int(w.cu_q[s]), int(w.cu_q[s + 1])
        o, l, _ = oracle.attn_paged(w.q_block[a:b], kp, vp, w.page_table[s], "f32", int(w.prefix_len[s]))
        assert np.array_equal(out[a:b], o) and np.array_equal(lse[a:b], l)


# ------------------------------------------------------------------ acceptance
def _kv(path):
    d = {}
    for line in open(path):
        line = line.strip()
        if not line or line.startswith("#"):
            continue
        k, v = line.split("=")
        d[k.strip()] = [int(x) for x in v.split()]
    return d


def test_accept_paper_worked_example():
    g = _kv(os.path.join(GOLDEN, "specdec_worked_example.txt"))
    V = 128
    k = g["n_drafts"][0]
    logits = np.zeros((k + 1, V), dtype=np.float32)
    for r, t in enumerate(g["target_tokens"]):
        logits[r, t] = 5.0
    am, al, nt, sl = oracle.accept_greedy(logits, "f32", V, g["drafts"], [0, k + 1], [100])
    assert al[0] == g["expected_accept_len"][0]
    assert nt[0] == g["expected_next_token"][0]
    emitted = list(g["drafts"][: al[0]]) + [int(nt[0])]
    assert emitted == g["expected_emitted"] and len(emitted) == g["expected_tokens_emitted"][0]
    assert sl[0] == 100 + 3 + 1


def test_argmax_matches_numpy_first_occurrence_with_real_ties():
    # bf16 N(0,1) logits over a big vocabulary tie at the top in a noticeable share of rows
    x = W.natural_logits(5, 64, 128256, "bf16")
    drafts = np.zeros(0, dtype=np.int32)
    cu = np.arange(65, dtype=np.int32)  # 64 sequences with q=1
    am, al, nt, sl = oracle.accept_greedy(x, "bf16", 128256, drafts, cu, np.zeros(64, np.int32))
    xf = W.bf16_bits_to_f32(x)
    ref = np.argmax(xf, axis=1)
    assert np.array_equal(am, ref) and np.array_equal(nt, ref) and np.all(al == 0)
    ties = sum(int((xf[r] == xf[r].max()).sum() > 1) for r in range(64))
    assert ties >= 1  # the tie rule is actually exercised


def test_argmax_tie_zero_sign_nan_inf_and_padding():
    V = 16
    x = np.full((6, V + 4), 9.0, dtype=np.float32)  # 4 padding columns hold a larger value
    x[:, :V] = -1.0
    x[0, [3, 7]] = 2.0                      # tie -> 3
    x[1, :V] = -0.0; x[1, 5] = 0.0          # -0 == +0: all tie -> 0
    x[2, :V] = np.nan; x[2, 9] = -50.0      # NaN never beats a number -> 9
    x[3, :V] = np.nan                       # all NaN -> 0
    x[4, :V] = -np.inf                      # all -inf tie -> 0
    x[5, 2] = np.inf; x[5, 1] = 1e30        # +inf wins -> 2
    cu = np.arange(7, dtype=np.int32)
    am, _, _, _ = oracle.accept_greedy(x, "f32", V, np.zeros(0, np.int32), cu, np.zeros(6, np.int32))
    assert am.tolist() == [3, 0, 9, 0, 0, 2]


def brute_accept(t_rows, drafts):
    a = 0
    for i, d in enumerate(drafts):
        if d != t_rows[i]:
            break
        a += 1
    return a, t_rows[a]


def test_accept_brute_force_all_small_cases():
    """Every draft pattern over a 3-token alphabet for k <= 4, against a literal loop."""
    import itertools
    V = 3
    for k in range(0, 5):
        for t_rows in itertools.product(range(V), repeat=k + 1):
            logits = np.zeros((k + 1, V), dtype=np.float32)
            for r, t in enumerate(t_rows):
                logits[r, t] = 1.0
            for drafts in itertools.product(range(V), repeat=k):
                am, al, nt, sl = oracle.accept_greedy(logits, "f32", V, np.array(drafts, np.int32), [0, k + 1], [7])
                a, nxt = brute_accept(t_rows, drafts)
                assert (int(al[0]), int(nt[0]), int(sl[0])) == (a, nxt, 7 + a + 1)


def test_accept_later_drafts_do_not_matter_and_plan_is_met():
    aw = W.make_planted_accept("t", 21, "bf16", 5000, [8, 1, 4, 16, 2], [10, 20, 30, 40, 50])
    am, al, nt, sl = oracle.accept_greedy(aw.logits, "bf16", aw.vocab, aw.drafts, aw.cu_q, aw.prefix_len)
    assert np.array_equal(am, aw.planted_targets)
    assert np.array_equal(al, aw.planned_accept)
    assert np.array_equal(sl, aw.prefix_len + al + 1)
    d2 = aw.drafts.copy()
    for s in range(5):  # scramble everything after the first mismatch
        k = int(aw.cu_q[s + 1] - aw.cu_q[s]) - 1
        base = int(aw.cu_q[s]) - s
        for i in range(int(al[s]) + 1, k):
            d2[base + i] = (d2[base + i] + 17) % aw.vocab
    am2, al2, nt2, sl2 = oracle.accept_greedy(aw.logits, "bf16", aw.vocab, d2, aw.cu_q, aw.prefix_len)
    assert np.array_equal(al, al2) and np.array_equal(nt, nt2)
    # out-of-range drafts are legal and simply never match
    d3 = np.full_like(aw.drafts, -5)
    _, al3, nt3, _ = oracle.accept_greedy(aw.logits, "bf16", aw.vocab, d3, aw.cu_q, aw.prefix_len)
    assert np.all(al3 == 0) and np.array_equal(nt3, aw.planted_targets[aw.cu_q[:-1]])


# ------------------------------------------------------------------ check 5: greedy equivalence
def test_check5_speculative_greedy_equals_token_by_token():
    from oracle.toy_lm import ToyLM, build_ngram_table, ngram_drafts
    from tests.spec_loop import OracleBackend, generate

    lm = ToyLM(seed=11)
    rng = np.random.default_rng(3)
    motif = rng.integers(0, lm.vocab, 12).tolist()
    prompt = (motif * 3 + rng.integers(0, lm.vocab, 5).tolist() + motif[:6])
    T = 48
    base, calls0, _ = generate(OracleBackend(lm), prompt, T)
    assert calls0 == T

    def right(history, k):  # always-right drafts: the true continuation
        n = len(history) - len(prompt)
        return (base + [0] * k)[n:n + k]

    def wrong(history, k):
        return [(t + 1) % lm.vocab for t in right(history, k)]

    table = build_ngram_table(prompt, 3)
    lut_rng = np.random.default_rng(9)

    def lut(history, k):
        return ngram_drafts(table, history, k, 3, lut_rng, lm.vocab)

    out_r, calls_r, acc_r = generate(OracleBackend(lm), prompt, T, right, k=4)
    out_w, calls_w, acc_w = generate(OracleBackend(lm), prompt, T, wrong, k=4)
    out_l, calls_l, acc_l = generate(OracleBackend(lm), prompt, T, lut, k=4)
    assert out_r == base and out_w == base and out_l == base
    assert all(a == 4 for a in acc_r[:-1]) and calls_r <= math.ceil(T / 5) + 1
    assert all(a == 0 for a in acc_w) and calls_w == T


def test_ngram_table_most_frequent_successor():
    from oracle.toy_lm import build_ngram_table, ngram_drafts
    stream = [1, 2, 3, 1, 2, 4, 1, 2, 4, 9, 9, 9]
    t = build_ngram_table(stream, 3)
    assert t[(1, 2)] == 4 and t[(9, 9)] == 9 and (2, 9) not in t
    assert build_ngram_table([5, 6, 8, 5, 6, 7], 3)[(5, 6)] == 7  # count tie: lowest token id
    assert build_ngram_table([5, 6, 7, 5, 6, 8], 3)[(5, 6)] == 7
    rng = np.random.default_rng(0)
    assert ngram_drafts(t, [7, 7], 4, 3, rng, 10) is None  # first lookup misses -> fallback
    d = ngram_drafts(t, [0, 1, 2], 3, 3, rng, 10)
    assert d[0] == 4 and d[1] == 1 and len(d) == 3  # (1,2)->4, (2,4)->1, (4,1)->2
    assert d[2] == 2


def _naive_ngram(stream, n):
    """Independent restatement with collections.Counter: most common successor, ties to the lowest id."""
    from collections import Counter, defaultdict
    succ = defaultdict(Counter)
    for w in zip(*[stream[i:] for i in range(n)]):
        succ[tuple(int(t) for t in w[:-1])][int(w[-1])] += 1
    return {k: sorted(c.items(), key=lambda kv: (-kv[1], kv[0]))[0][0] for k, c in succ.items()}


@pytest.mark.parametrize("n", [1, 2, 3, 4])
def test_ngram_table_against_counter_brute_force(n):
    from oracle.toy_lm import build_ngram_table
    rng = np.random.default_rng(100 + n)
    for length, alphabet in [(0, 3), (n - 1, 3), (n, 3), (50, 2), (400, 5), (3000, 40)]:
        stream = rng.integers(0, alphabet, size=max(length, 0)).tolist()
        assert build_ngram_table(stream, n) == _naive_ngram(stream, n)


def test_ngram_drafts_reproduce_a_periodic_stream_and_fall_back_on_unknown_context():
    """Closed form: on a stream that repeats a block of distinct tokens every bigram has one successor, so
    the trigram chain continues the stream exactly; an unseen context gives no drafts at all (Sec. 4.3,
    selective decoding), a context that goes unknown mid-chain takes the supplied guesses."""
    from oracle.toy_lm import build_ngram_table, ngram_drafts
    block = [11, 4, 7, 300, 2, 9]
    stream = block * 5
    t = build_ngram_table(stream, 3)
    assert len(t) == len(block)
    assert ngram_drafts(t, stream[:8], 9, 3, fill=[0] * 9) == (block * 4)[8 % 6:8 % 6 + 9]
    assert ngram_drafts(t, [4, 11], 3, 3, fill=[0] * 3) is None
    open_ended = build_ngram_table([1, 2, 3, 4], 3)          # (1,2)->3, (2,3)->4, nothing after (3,4)
    assert ngram_drafts(open_ended, [1, 2], 4, 3, fill=[50, 51, 52, 53]) == [3, 4, 52, 53]
    assert ngram_drafts(build_ngram_table([5, 5, 6, 5, 7, 5, 6], 2), [5], 2, 2, fill=[0, 0]) == [6, 5]  # bigram: 5 -> 6 twice
