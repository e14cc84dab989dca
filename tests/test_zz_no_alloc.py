"""klpm_select_noalloc: the selection entry point for hosts that forbid device allocations.

An inference server that pre-allocates the whole GPU for its own pool, or a scheduler tick that must not
hit the implicit synchronisation of cudaMalloc, cannot use klpm_select (it allocates its reduction scratch
on first use).  The no-alloc variant keeps that scratch in a fixed array inside the library.  This file
checks, through the C ABI, that it returns exactly the pick klpm_select returns -- picks are indices, so the
comparison is exact -- on two calls in a row that share the fixed array, and that a queue longer than the
stated maximum is refused.  It is collected last on purpose: a failure here cannot hide another test.
"""
import ctypes

import pytest
import torch

pytestmark = pytest.mark.gpu


def _case(seed, n):
    g = torch.Generator().manual_seed(seed)
    m = torch.randint(0, 5, (n,), generator=g, dtype=torch.int32).cuda()
    t = (torch.randint(0, 40, (n,), generator=g, dtype=torch.int64) * (1 << 34)).cuda()
    w = (torch.rand(n, generator=g) < 0.6).to(torch.uint8).cuda()
    return m, t, w


def test_noalloc_select_matches_select_on_consecutive_calls():
    from paper_2502_04677_b200 import binding as K
    want = torch.zeros(1, dtype=torch.int32, device="cuda")
    got = torch.zeros(1, dtype=torch.int32, device="cuda")
    first = _case(1, 600_000)
    torch.cuda.synchronize()
    free_before = torch.cuda.mem_get_info()[0]
    K.klpm_select_noalloc(*first, 1, K.make_params(K.POLICY_KLPM, 3), got)      # its first call on the device: set-up included
    torch.cuda.synchronize()
    assert torch.cuda.mem_get_info()[0] == free_before                          # the device's free memory has not moved
    # two calls back to back on the shared scratch, then more shapes: one block, many blocks, every kind of turn
    cases = [(1, 600_000, K.POLICY_KLPM, 3, 1), (2, 600_000, K.POLICY_KLPM, 3, 3), (3, 1, K.POLICY_LPM, 1, 0),
             (4, 2049, K.POLICY_FCFS, 1, 5), (5, 70_001, K.POLICY_KLPM, 2, 7), (6, 1000, K.POLICY_KLPM, 4, 8)]
    for seed, n, policy, k, counter in cases:
        m, t, w = _case(seed, n)
        p = K.make_params(policy, k)
        got.fill_(-5)
        K.klpm_select_noalloc(m, t, w, counter, p, got)
        K.klpm_select(m, t, w, counter, p, want)
        assert int(got.item()) == int(want.item()), (seed, n, policy, k, counter)
        assert int(want.item()) >= 0
    # nobody waiting -> -1 from both
    m, t, w = _case(9, 5000)
    w.zero_()
    K.klpm_select_noalloc(m, t, w, 1, K.make_params(K.POLICY_LPM), got)
    K.klpm_select(m, t, w, 1, K.make_params(K.POLICY_LPM), want)
    assert int(got.item()) == int(want.item()) == -1


def test_noalloc_select_rejects_queues_above_its_limit():
    from paper_2502_04677_b200 import binding as K
    m, t, w = _case(1, 16)
    pick = torch.full((1,), -9, dtype=torch.int32, device="cuda")
    # straight through the C ABI: only the stated length is above the limit, and nothing may be read for it
    p = K.make_params(K.POLICY_LPM)
    vp = lambda x: ctypes.c_void_p(x.data_ptr())
    rc = K.lib().klpm_select_noalloc(vp(m), vp(t), vp(w), K.SELECT_NOALLOC_MAX_QUERIES + 1, 0, ctypes.byref(p), vp(pick),
                                     ctypes.c_void_p(torch.cuda.current_stream().cuda_stream))
    assert rc == K.RT_ERR_TOO_LARGE
    with pytest.raises(ValueError):
        K.klpm_select_noalloc(m, t[:8], w, 0, p, pick)                           # the three arrays must agree in length
    torch.cuda.synchronize()
    assert int(pick.item()) == -9          # nothing was launched
