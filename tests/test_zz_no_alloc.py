"""agx_accept_greedy_static: the accept step for callers that cannot allocate device memory
(a runtime living in a fixed arena, or code next to an allocator it must not touch).  It takes no
handle and no workspace; its scratch is a fixed array inside the library.  The tests call it through
the C ABI, several calls in a row on the shared array, and require the integers of the CPU oracle
(and therefore those of agx_accept_greedy with a workspace, which is checked against the oracle too).

Collected last on purpose (file name), so a run that stops at the first failure has already run
every other test.
"""
import numpy as np
import pytest
import torch

import oracle
from paper_2605_10380_b200 import agx
from paper_2605_10380_b200 import workloads as W
from tests.gpu_util import dev, run_accept

pytestmark = pytest.mark.gpu


def run_static(aw):
    logits = dev(aw.logits, aw.dtype)
    drafts = dev(aw.drafts) if aw.drafts.size else torch.zeros(1, dtype=torch.int32, device="cuda")
    cu_q = dev(aw.cu_q)
    B = len(aw.cu_q) - 1
    rows = int(aw.cu_q[-1])
    acc = torch.full((B,), -7, dtype=torch.int32, device="cuda")
    nxt = torch.full((B,), -7, dtype=torch.int32, device="cuda")
    am = torch.full((rows,), -7, dtype=torch.int32, device="cuda")
    sl = dev(aw.prefix_len.copy())
    agx.accept_greedy_static(logits[:rows], aw.dtype, aw.vocab, drafts, cu_q, acc, nxt, am, sl)
    torch.cuda.synchronize()
    return am.cpu().numpy(), acc.cpu().numpy(), nxt.cpu().numpy(), sl.cpu().numpy()


def oracle_accept(aw):
    return oracle.accept_greedy(aw.logits, aw.dtype, aw.vocab, aw.drafts, aw.cu_q, aw.prefix_len)


def same(got, want, what):
    for name, g, w_ in zip(("argmax", "accept_len", "next_token", "seq_lens"), got, want):
        assert np.array_equal(g, w_), f"{what}: {name} differs"


def test_static_accept_matches_oracle_and_workspace_accept_on_calls_in_a_row():
    h = agx.Handle(32, 8, 128, "bf16")
    first = W.make_planted_accept("static_a", 61, "bf16", 128256, [8, 1, 4, 16], [4096, 10, 777, 2048])
    second = W.make_planted_accept("static_b", 62, "f32", 5003, [3] * 40 + [1] * 7, np.arange(47) * 3, row_stride=5008)
    for aw in (first, second, first):  # calls in a row share the library's scratch array, shapes alternate
        want = oracle_accept(aw)
        same(run_static(aw), want, aw.name)
        same(run_accept(h, aw), want, aw.name + " (workspace variant)")


def test_static_accept_natural_ties_against_oracle():
    """bf16 N(0,1) logits over the full vocabulary carry real ties at the top: lowest index must win."""
    rng = np.random.default_rng(63)
    logits = W.natural_logits(63, 24, 128256, "bf16")
    values = (logits.astype(np.uint32) << 16).view(np.float32)
    assert any(int((row == row.max()).sum()) > 1 for row in values), "the seed no longer produces a tie at the top"
    cu = W.cu_from_q([8, 8, 8])
    am = oracle.accept_greedy(logits, "bf16", 128256, np.zeros(21, np.int32), cu, np.zeros(3, np.int32))[0]
    drafts = np.concatenate([am[0:7], am[8:12], rng.integers(0, 128256, 3), am[16:17], [am[17] + 1], am[18:23]]).astype(np.int32)
    aw = W.AcceptWorkload("static_ties", "bf16", 128256, 128256, logits, drafts, cu, np.array([5, 6, 7], np.int32))
    want = oracle_accept(aw)
    assert want[1].tolist() == [7, 4, 1]
    same(run_static(aw), want, "ties")
    same(run_static(aw), want, "ties, second call")


def test_static_accept_at_its_row_limit():
    """Exactly 2048 logits rows (the fixed scratch holds no more): 256 sequences of 8 rows over a
    32768-entry vocabulary, twice, against the oracle."""
    aw = W.make_planted_accept("static_2048", 64, "bf16", 32768, [8] * 256, np.arange(256) * 5)
    assert int(aw.cu_q[-1]) == 2048
    want = oracle_accept(aw)
    same(run_static(aw), want, "2048 rows")
    same(run_static(aw), want, "2048 rows, second call")


def test_static_accept_rejects_bad_sizes_and_misaligned_pointers():
    lib = agx.load()
    dummy = torch.zeros(64, dtype=torch.int32, device="cuda")
    stream = torch.cuda.current_stream().cuda_stream
    p = dummy.data_ptr()
    st = lib.agx_accept_greedy_static(p, agx.AGX_F32, 4, 4, p, p, 1, 2049, p, p, None, None, stream)
    assert st == -2  # AGX_E_RANGE: more than 2048 rows
    # misaligned pointers are argument errors (AGX_E_INVAL), never a device fault
    assert lib.agx_accept_greedy_static(p + 2, agx.AGX_F32, 4, 4, p, p, 1, 2, p, p, None, None, stream) == -1
    assert lib.agx_accept_greedy_static(p + 1, agx.AGX_BF16, 8, 8, p, p, 1, 2, p, p, None, None, stream) == -1
    assert lib.agx_accept_greedy_static(p, agx.AGX_F32, 4, 4, p + 2, p, 1, 2, p, p, None, None, stream) == -1
    assert lib.agx_accept_greedy_static(p, agx.AGX_F32, 4, 4, p, p, 1, 2, p + 2, p, None, None, stream) == -1
    assert lib.agx_accept_greedy_static(p, agx.AGX_F32, 4, 4, p, p, 1, 2, p, p, p + 2, None, stream) == -1
    torch.cuda.synchronize()
