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
