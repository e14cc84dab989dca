"""The five configurations at their full size, in the launch configuration bench.py times: every output
array of the CUDA library is compared with the CPU oracle's through SHA-256 digests of the whole arrays
(bit-exact or not at all) plus a stored sample of values.  The expected digests are in tests/golden/
fullsize_<config>.json, written by tests/golden/make_fullsize_golden.py, which calls only the oracle."""
import hashlib
import json
import os

import numpy as np
import pytest
import torch

from paper_2502_04677_b200 import workloads as W

pytestmark = pytest.mark.gpu
GOLDEN = os.path.join(os.path.dirname(__file__), "golden")


def digest(t: torch.Tensor, dtype: str) -> str:
    return hashlib.sha256(np.ascontiguousarray(t.cpu().numpy().astype(dtype)).tobytes()).hexdigest()


@pytest.mark.parametrize("name", ["tiny", "medium", "hierarchical", "streaming", "adversarial"])
def test_full_size_configuration_is_bit_exact(name):
    path = os.path.join(GOLDEN, "fullsize_%s.json" % name)
    if not os.path.exists(path):
        pytest.skip("no stored oracle digests for %s" % name)
    g = json.load(open(path))
    import bench
    from paper_2502_04677_b200 import binding as K
    w = W.WORKLOADS[name]() if name == "tiny" else W.WORKLOADS[name](scale=1.0)
    assert w.queries.n == g["queries"] and w.prefill.n == g["prefill"] and w.recipe == g["recipe"]
    device = torch.device("cuda", 0)
    tree, q_tok, q_off, arr = bench.device_workload(w, device)
    st = K.rt_stats(tree)
    for key in ("n_nodes", "tokens", "clock"):
        assert st[key] == g["tree"][key], key
    nq = w.queries.n
    m = torch.zeros(nq, dtype=torch.int32, device=device)
    K.rt_match_batch(tree, q_tok, q_off, m)
    assert K.rt_sync_status(tree) == 0
    assert m[::g["match_len"]["sample_step"]].tolist() == g["match_len"]["sample"]
    assert int(m.sum(dtype=torch.int64)) == g["match_len"]["sum"]
    assert digest(m, "<i4") == g["match_len"]["sha256"]
    for key, want in g.get("schedule", {}).items():
        label, k = key.split("_k")
        policy = {"klpm": K.POLICY_KLPM, "fcfs": K.POLICY_FCFS, "lpm": K.POLICY_LPM}[label]
        K.rt_rollback(tree)
        order = torch.full((nq,), -1, dtype=torch.int32, device=device)
        unc = torch.full((nq,), -1, dtype=torch.int32, device=device)
        ttft = torch.full((nq,), -1, dtype=torch.int64, device=device)
        comp = torch.full((nq,), -1, dtype=torch.int64, device=device)
        K.klpm_run(tree, q_tok, q_off, arr, K.make_params(policy, int(k), 0, 1, w.start_tick), order, unc, ttft, comp)
        assert K.rt_sync_status(tree) == 0, key
        assert order[:16].tolist() == want["order_head"] and order[-16:].tolist() == want["order_tail"], key
        assert int(unc.sum(dtype=torch.int64)) == want["total_uncached"], key
        assert digest(order, "<i4") == want["order_sha256"], key
        assert digest(unc, "<i4") == want["uncached_sha256"], key
        assert digest(ttft, "<i8") == want["ttft_sha256"], key
        assert digest(comp, "<i8") == want["completion_sha256"], key
        after = K.rt_stats(tree)
        for f in ("n_nodes", "tokens", "clock", "evictions"):
            assert after[f] == want["tree_after"][f], (key, f)
    K.rt_destroy(tree)


def test_adversarial_full_size_properties_and_both_loops():
    """The bench's own configuration (262,144 queries, k = 4) is too large for the CPU oracle's schedule, so the
    scheduling loop is checked there through what holds at any size -- the order is a permutation; every k-th
    decision takes the oldest unprocessed query (everybody is waiting); every other decision takes a query whose
    uncached-token count is consistent with its stored match; the uncached tokens add up to the growth of the
    tree; completion times are the running sum of the uncached tokens (1 tick per token) and TTFT = completion -
    arrival -- and through bit-exact agreement of the two device loops (the one-by-one loop is the one the oracle
    checks at the smaller sizes)."""
    import bench
    from paper_2502_04677_b200 import binding as K
    w = W.adversarial(scale=1.0)
    device = torch.device("cuda", 0)
    tree, q_tok, q_off, arr = bench.device_workload(w, device)
    nq, k = w.queries.n, 4
    before = K.rt_stats(tree)
    outs = []
    for legacy in (False, True):
        K.klpm_debug_set("run_one_by_one", 1 if legacy else 0)
        K.rt_rollback(tree)
        order = torch.full((nq,), -1, dtype=torch.int32, device=device)
        unc = torch.full((nq,), -1, dtype=torch.int32, device=device)
        ttft = torch.full((nq,), -1, dtype=torch.int64, device=device)
        comp = torch.full((nq,), -1, dtype=torch.int64, device=device)
        K.klpm_run(tree, q_tok, q_off, arr, K.make_params(K.POLICY_KLPM, k, 0, 1, w.start_tick), order, unc, ttft, comp)
        assert K.rt_sync_status(tree) == 0
        assert K.klpm_run_path(tree) == (K.RUN_PATH_ONE_BY_ONE if legacy else K.RUN_PATH_GROUPED)
        outs.append((order.cpu(), unc.cpu(), ttft.cpu(), comp.cpu(), K.rt_stats(tree)))
    K.klpm_debug_set("run_one_by_one", -1)
    order, unc, ttft, comp, after = outs[0]
    for a, b in zip(outs[0][:4], outs[1][:4]):
        assert torch.equal(a, b)
    assert {f: outs[0][4][f] for f in ("n_nodes", "tokens", "clock")} == {f: outs[1][4][f] for f in ("n_nodes", "tokens", "clock")}
    o = order.numpy().astype(np.int64)
    assert np.array_equal(np.sort(o), np.arange(nq))
    # everybody has arrived (start_tick = last arrival): the oldest unprocessed query by (arrival, index)
    a = arr.cpu().numpy()
    rank = np.empty(nq, dtype=np.int64)
    rank[np.lexsort((np.arange(nq), a))] = np.arange(nq)
    done = np.zeros(nq, dtype=bool)
    by_rank = np.argsort(rank)
    ptr = 0
    for c in range(nq):
        if c % k == 0:
            while done[by_rank[ptr]]:
                ptr += 1
            assert o[c] == by_rank[ptr], c
        done[o[c]] = True
    u = unc.numpy().astype(np.int64)
    lens = (q_off[1:] - q_off[:-1]).cpu().numpy()
    assert np.all(u >= 0) and np.all(u <= lens)
    assert int(u.sum()) == after["tokens"] - before["tokens"]
    assert after["clock"] == before["clock"] + nq
    cm = comp.numpy()
    assert np.array_equal(cm[o], w.start_tick + np.cumsum(u[o]))
    assert np.array_equal(ttft.numpy(), cm - a)
    K.rt_destroy(tree)
