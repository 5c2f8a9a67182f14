"""ep_reorder_static: the permutation for callers that cannot allocate device memory.

A plug-in running inside another framework, a process whose device memory was all handed out at
start-up, or a loop that cannot afford cudaMalloc's device-wide synchronisation has no way to give
ep_reorder a workspace or even to create a context.  ep_reorder_static keeps its scratch in an array
compiled into the library instead.  These tests call it through the C ABI and require the same
permutation, bit for bit, as the ordinary entry point and as the CPU oracle's stable counting sort
(integer outputs are compared exactly everywhere in this suite) -- twice in a row, because the
second call starts from whatever the first one left in the shared scratch.

This file sorts last on purpose: a run that stops at the first failure has then already executed
every other test.
"""
import ctypes

import numpy as np
import pytest
import torch

import oracle


def _labels(N, K, seed):
    g = torch.Generator().manual_seed(seed)
    return torch.randint(0, K, (N,), generator=g, dtype=torch.int32)


def test_sizes_beyond_the_built_in_scratch_are_refused_on_the_host():
    """No GPU needed: the limits are checked before the first CUDA call."""
    from paper_2604_01000_b200 import binding
    lib = binding.load_library()
    buf = (ctypes.c_int32 * 4)()
    p = ctypes.cast(buf, ctypes.c_void_p)
    too_many = binding.REORDER_STATIC_MAX_N + 1
    assert lib.ep_reorder_static(p, too_many, 4, p, None, None, None) == 2            # EP_ERR_UNSUPPORTED
    assert lib.ep_reorder_static(p, 4, binding.REORDER_STATIC_MAX_K + 1, p, None, None, None) == 2
    assert lib.ep_reorder_static(None, 4, 2, p, None, None, None) == 1                # EP_ERR_INVALID_ARG
    assert lib.ep_reorder_static(p, 0, 2, p, None, None, None) == 1
    assert lib.ep_status_string(2) == b"unsupported device or shape"


@pytest.mark.gpu
def test_two_calls_in_a_row_match_the_workspace_entry_point():
    import paper_2604_01000_b200 as ep
    ctx = ep.Context(0)
    status = torch.full((1,), -1, dtype=torch.int32, device="cuda")
    # the second case is smaller and has other labels, so stale counts from the first would show
    for N, K, seed in ((1_000_003, 64, 11), (250_007, 256, 12), (4097, 3, 13)):
        assign = _labels(N, K, seed).cuda()
        if K > 3:
            assign[assign == 2] = 3                                                    # an empty partition
        want = ctx.reorder(assign, K)
        got = ep.ep_reorder_static(assign, K, status=status)
        torch.cuda.synchronize()
        assert int(status.item()) == 0
        assert torch.equal(got.perm, want.perm)
        assert torch.equal(got.inv_perm, want.inv_perm)
        perm, inv = oracle.reorder(assign.cpu().numpy(), K)                            # and the definition itself
        np.testing.assert_array_equal(got.perm.cpu().numpy(), perm)
        np.testing.assert_array_equal(got.inv_perm.cpu().numpy(), inv)
        again = ep.ep_reorder_static(assign, K, inverse=False)                         # same input, scratch now dirty
        torch.cuda.synchronize()
        assert again.inv_perm is None and torch.equal(again.perm, want.perm)
    ctx.check()
    ctx.close()


@pytest.mark.gpu
def test_bad_label_is_reported_through_the_status_word_and_the_next_call_is_clean():
    import paper_2604_01000_b200 as ep
    status = torch.zeros(1, dtype=torch.int32, device="cuda")
    ep.ep_reorder_static(torch.tensor([0, 5, 1], dtype=torch.int32).cuda(), 2, status=status)
    torch.cuda.synchronize()
    assert int(status.item()) == 4                                                     # EP_ERR_BAD_INDEX
    good = torch.tensor([1, 0, 1, 0], dtype=torch.int32).cuda()
    r = ep.ep_reorder_static(good, 2, status=status)
    torch.cuda.synchronize()
    assert int(status.item()) == 0
    assert r.perm.tolist() == [1, 3, 0, 2] and r.inv_perm.tolist() == [2, 0, 3, 1]
