"""agx_accept_greedy_static: the accept step for callers that cannot allocate device memory
(a runtime living in a fixed arena, or code next to an allocator it must not touch).  It takes no
handle and no workspace; its scratch is a fixed array inside the library.  The test calls it through
the C ABI twice in a row and requires the same integers as agx_accept_greedy with a workspace.

Collected last on purpose (file name), so a run that stops at the first failure has already run
every other test.
"""
import numpy as np
import pytest
import torch

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


def test_static_accept_matches_workspace_accept_twice_in_a_row():
    h = agx.Handle(32, 8, 128, "bf16")
    first = W.make_planted_accept("static_a", 61, "bf16", 128256, [8, 1, 4, 16], [4096, 10, 777, 2048])
    second = W.make_planted_accept("static_b", 62, "f32", 5003, [3] * 40 + [1] * 7, np.arange(47) * 3, row_stride=5008)
    for aw in (first, second):  # two calls in a row share the library's scratch array
        want = run_accept(h, aw)
        got = run_static(aw)
        for g, w_ in zip(got, want):
            assert np.array_equal(g, w_)
    # and the first problem again, after the scratch was used by a different shape
    for g, w_ in zip(run_static(first), run_accept(h, first)):
        assert np.array_equal(g, w_)


def test_static_accept_rejects_sizes_beyond_its_fixed_scratch():
    lib = agx.load()
    dummy = torch.zeros(16, dtype=torch.int32, device="cuda")
    st = lib.agx_accept_greedy_static(dummy.data_ptr(), agx.AGX_F32, 4, 4, dummy.data_ptr(), dummy.data_ptr(),
                                      1, 2049, dummy.data_ptr(), dummy.data_ptr(), None, None,
                                      torch.cuda.current_stream().cuda_stream)
    assert st == -2  # AGX_E_RANGE: more than 2048 rows
