"""The grouped scheduling loop (trees without a budget) against the oracle and against the one-by-one loop.

klpm_run on a tree without a budget keeps every query's match state itself: queries whose match ends at the
same tree position and continues with the same token form a group, and processing a prompt re-matches its
group only.  These cases aim at the group machinery: groups of 2..32 (one warp), groups up to 4,096 (sorted in
shared memory), larger groups (kept together), queries that have not arrived when their group changes,
identical prompts, prompts that are prefixes of others, and the tie-priority / hit-rate variants."""
import numpy as np
import pytest
import torch

import oracle
from paper_2502_04677_b200 import workloads as W

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def K():
    from paper_2502_04677_b200 import binding
    return binding


def dev(t):
    return t.cuda() if isinstance(t, torch.Tensor) else torch.as_tensor(t).cuda()


def run_gpu(K, prefill, prompts, arr, policy, k, prio=None, score_mode=0, start=0, c_num=0, c_den=1, legacy=False,
            from_match=False):
    pt, po = W.to_csr(prefill)
    qt, qo = W.to_csr(prompts)
    n, npre = len(prompts), len(prefill)
    cap = dict(max_nodes=2 * (n + npre) + 16, max_pool_tokens=pt.numel() + qt.numel() + 8 * (n + npre) + 16,
               max_clock=n + npre + 16)
    tree = K.rt_build(dev(pt), dev(po), **cap) if npre else K.rt_create(**cap)
    order = torch.full((n,), -1, dtype=torch.int32, device="cuda")
    unc = torch.full((n,), -1, dtype=torch.int32, device="cuda")
    ttft = torch.full((n,), -1, dtype=torch.int64, device="cuda")
    comp = torch.full((n,), -1, dtype=torch.int64, device="cuda")
    d_prio = None if prio is None else dev(torch.as_tensor(prio, dtype=torch.int64))
    K.klpm_debug_set("run_one_by_one", 1 if legacy else 0)
    d_qt, d_qo = dev(qt), dev(qo)
    state = None
    if from_match:       # the loop starts from the records of a batched match instead of walking the queries itself
        state = K.match_state_buffer(n, "cuda")
        m0 = torch.zeros(n, dtype=torch.int32, device="cuda")
        K.rt_match_batch_ex(tree, d_qt, d_qo, m0, None, None, state)
    try:
        K.klpm_run_ex(tree, d_qt, d_qo, dev(torch.as_tensor(arr, dtype=torch.int64)),
                      K.make_params(policy, k, c_num, c_den, start), d_prio, score_mode, order, unc, ttft, comp, state)
    finally:
        K.klpm_debug_set("run_one_by_one", -1)
    assert K.rt_sync_status(tree) == 0
    assert K.klpm_run_path(tree) == (K.RUN_PATH_ONE_BY_ONE if legacy else K.RUN_PATH_GROUPED)
    st = K.rt_stats(tree)
    # the grown tree answers matches like the oracle's: every processed prompt is fully cached
    m = torch.zeros(n, dtype=torch.int32, device="cuda")
    K.rt_match_batch(tree, dev(qt), dev(qo), m)
    assert K.rt_sync_status(tree) == 0
    assert np.array_equal(m.cpu().numpy(), (qo[1:] - qo[:-1]).numpy())
    K.rt_destroy(tree)
    return order.cpu().numpy(), unc.cpu().numpy(), ttft.cpu().numpy(), comp.cpu().numpy(), st


def run_oracle(prefill, prompts, arr, policy, k, prio=None, score_mode=0, start=0, c_num=0, c_den=1,
               tier=oracle.TIER_UPDATE):
    pt, po = W.to_csr(prefill)
    qt, qo = W.to_csr(prompts)
    ot = oracle.OracleTree(0)
    if len(prefill):
        ot.insert(pt.numpy(), po.numpy())
    out = oracle.schedule(qt.numpy(), qo.numpy(), np.asarray(arr, dtype=np.int64), policy, k, c_num, c_den, start,
                          oracle.CACHE_TREE, tier, ot, prio, score_mode)
    return out + (ot.stats(),)


def same(got, want):
    for g, w, name in zip(got[:4], want[:4], ("order", "uncached", "ttft", "completion")):
        assert np.array_equal(g, w), name
    for key in ("n_nodes", "tokens", "clock"):
        assert got[4][key] == want[4][key], key


def shared_prefix_queue(seed, n, levels, tail, vocab, max_gap):
    """Prompts = one block per level (each level has a few alternatives, so many prompts tie at every depth)
    + a short random tail over a small alphabet; arrival gaps in [0, max_gap]."""
    rng = np.random.RandomState(seed)
    blocks = [[rng.randint(0, vocab, size=ln).tolist() for _ in range(alts)] for ln, alts in levels]
    prompts, arr, t = [], [], 0
    for _ in range(n):
        p = []
        for alts in blocks:
            p += alts[rng.randint(len(alts))]
        p += rng.randint(0, vocab, size=rng.randint(0, tail + 1)).tolist()
        prompts.append(p)
        t += int(rng.randint(0, max_gap + 1))
        arr.append(t)
    return prompts, arr


@pytest.mark.parametrize("seed", range(3))
@pytest.mark.parametrize("max_gap", [0, 40])
def test_groups_of_every_size_small_queue(K, seed, max_gap):
    """300 prompts over 3 levels of shared blocks and a binary tail: groups from 2 to ~150 members, identical
    prompts, prompts that are prefixes of others; with gaps, members join their groups before they arrive."""
    prompts, arr = shared_prefix_queue(seed, 300, [(6, 2), (5, 3), (4, 2)], tail=6, vocab=2, max_gap=max_gap)
    prefill, _ = shared_prefix_queue(seed + 77, 10, [(6, 2), (5, 3)], tail=3, vocab=2, max_gap=0)
    for policy, k in ((0, 1), (1, 1), (2, 2), (2, 5)):
        got = run_gpu(K, prefill, prompts, arr, policy, k, c_num=1, c_den=3)
        want = run_oracle(prefill, prompts, arr, policy, k, c_num=1, c_den=3, tier=oracle.TIER_REMATCH)
        same(got, want)


@pytest.mark.parametrize("max_gap", [0, 3])
def test_groups_sorted_in_shared_memory(K, max_gap):
    """3,000 prompts, empty tree: the first pick dissolves a group of ~1,500 (sorted inside the CTA), which
    splits into groups of hundreds, and so on down to single queries."""
    prompts, arr = shared_prefix_queue(5, 3000, [(12, 2), (9, 4), (7, 5)], tail=8, vocab=3, max_gap=max_gap)
    for policy, k in ((1, 1), (2, 3)):
        got = run_gpu(K, [], prompts, arr, policy, k)
        want = run_oracle([], prompts, arr, policy, k)
        same(got, want)


@pytest.mark.parametrize("max_gap", [0, 2])
def test_groups_too_large_to_sort(K, max_gap):
    """6,000 prompts that all start with the same block: the first group has ~6,000 members (more than the CTA
    sorts), so it stays one run whose members are checked one by one until it has shrunk."""
    prompts, arr = shared_prefix_queue(9, 6000, [(10, 1), (8, 3), (6, 4)], tail=5, vocab=4, max_gap=max_gap)
    got = run_gpu(K, [], prompts, arr, K.POLICY_KLPM, 4)
    want = run_oracle([], prompts, arr, oracle.POLICY_KLPM, 4)
    same(got, want)


@pytest.mark.parametrize("score_mode", [0, 1])
def test_grouped_loop_with_priorities_and_hit_rate(K, score_mode):
    prompts, arr = shared_prefix_queue(21, 500, [(5, 2), (4, 3)], tail=7, vocab=2, max_gap=6)
    prio = np.random.RandomState(3).randint(0, 50, size=len(prompts)).tolist()
    for policy, k in ((1, 1), (2, 3)):
        got = run_gpu(K, [], prompts, arr, policy, k, prio=prio, score_mode=score_mode)
        want = run_oracle([], prompts, arr, policy, k, prio=prio, score_mode=score_mode, tier=oracle.TIER_REMATCH)
        same(got, want)


@pytest.mark.parametrize("score_mode", [0, 1])
def test_list_mode_with_priorities_all_waiting(K, score_mode):
    """Everybody waiting from the start, mostly distinct continuations, random tie priorities: the loop works from
    the presorted key list in warp-wide steps, with key ranks that are not the slots."""
    rng = np.random.RandomState(11)
    prefixes = [rng.randint(0, 50, size=ln).tolist() for ln in (20, 35, 35, 50, 64)]
    prompts = [prefixes[rng.randint(5)] + rng.randint(0, 5000, size=rng.randint(1, 30)).tolist() for _ in range(4000)]
    prefill = [p + [7] for p in prefixes[:4]]
    arr = [0] * len(prompts)
    prio = rng.randint(0, 1000, size=len(prompts)).tolist()
    for policy, k in ((1, 1), (2, 3), (2, 7)):
        got = run_gpu(K, prefill, prompts, arr, policy, k, prio=prio, score_mode=score_mode)
        want = run_oracle(prefill, prompts, arr, policy, k, prio=prio, score_mode=score_mode)
        same(got, want)


@pytest.mark.parametrize("n", [1, 31, 33, 100, 1000, 5001])
def test_list_mode_many_turn_patterns(K, n):
    """Everybody waiting, a tree that already holds the shared prefixes, mostly distinct continuations with a few
    identical prompts and a few shared continuations: warp-wide steps of every size and turn pattern (k below,
    at and above 32, k = 1, pure policies), queue lengths around the 32-lane boundaries."""
    rng = np.random.RandomState(100 + n)
    prefixes = [rng.randint(0, 1000, size=ln).tolist() for ln in (3, 17, 40, 40, 90)]
    prompts = []
    for _ in range(n):
        p = prefixes[rng.randint(5)] + rng.randint(0, 300, size=rng.randint(0, 12)).tolist()
        prompts.append(prompts[rng.randint(len(prompts))] if prompts and rng.rand() < 0.03 else p)
    prefill = [p + [1001] for p in prefixes]
    arr = [0] * n
    for policy, k in ((0, 1), (1, 1), (2, 1), (2, 2), (2, 3), (2, 5), (2, 31), (2, 32), (2, 33), (2, 1000)):
        got = run_gpu(K, prefill, prompts, arr, policy, k, c_num=1, c_den=2)
        want = run_oracle(prefill, prompts, arr, policy, k, c_num=1, c_den=2)
        same(got, want)


@pytest.mark.parametrize("name,scale,k", [("medium", 1 / 16, 4), ("adversarial", 1 / 256, 4), ("tiny", 1, 2)])
def test_both_loops_agree(K, name, scale, k):
    """The grouped loop and the one-by-one loop (forced by the debug setting run_one_by_one) give identical schedules."""
    w = W.tiny() if name == "tiny" else W.WORKLOADS[name](scale=scale)
    pt, po = w.prefill.materialize()
    qt, qo = w.queries.materialize()
    prefill = [pt[po[i]:po[i + 1]].tolist() for i in range(po.numel() - 1)]
    prompts = [qt[qo[i]:qo[i + 1]].tolist() for i in range(qo.numel() - 1)]
    a = run_gpu(K, prefill, prompts, w.arrivals, K.POLICY_KLPM, k, start=w.start_tick)
    b = run_gpu(K, prefill, prompts, w.arrivals, K.POLICY_KLPM, k, start=w.start_tick, legacy=True)
    same(a, b)


@pytest.mark.parametrize("max_blocks,smem_kb,n,max_gap", [(16, 0, 3000, 2), (4, 60, 3000, 2), (1, 0, 3000, 2), (4, 49, 3000, 0),
                                                         (16, 52, 20000, 0), (64, 49, 20000, 1)])
def test_large_queue_layout_on_a_small_queue(K, max_blocks, smem_kb, n, max_gap):
    """Queues above 262,144 use larger tournament leaf blocks and keep the two extra bitmaps of list mode -- far
    larger ones the processed bitmap too -- in global memory.  Shrinking the limits makes small streams take those
    paths: 64 to 4,096 slots per leaf block; every bitmap in shared memory, only the processed one, or none; with
    everybody waiting from the start (list mode throughout) and with arrivals over time."""
    K.klpm_debug_set("fast_max_blocks", max_blocks)
    K.klpm_debug_set("fast_smem_kb", smem_kb)
    try:
        prompts, arr = shared_prefix_queue(31, n, [(12, 3), (9, 4)], tail=9, vocab=5, max_gap=max_gap)
        prefill, _ = shared_prefix_queue(32, 200, [(12, 3), (9, 4)], tail=4, vocab=5, max_gap=0)
        for policy, k in ((2, 4), (0, 1), (1, 1)):
            got = run_gpu(K, prefill, prompts, arr, policy, k)
            want = run_oracle(prefill, prompts, arr, policy, k)
            same(got, want)
    finally:
        K.klpm_debug_set("fast_max_blocks", -1)
        K.klpm_debug_set("fast_smem_kb", -1)


def test_list_mode_all_arrived(K):
    """Everybody waiting from the start and mostly distinct continuations: the loop works from the presorted key
    list in warp-wide steps, cut short by the few grouped queries (medium at 1/8: 4,096 queries, 64 prefixes)."""
    w = W.medium(scale=1 / 8)
    pt, po = w.prefill.materialize()
    qt, qo = w.queries.materialize()
    prefill = [pt[po[i]:po[i + 1]].tolist() for i in range(po.numel() - 1)]
    prompts = [qt[qo[i]:qo[i + 1]].tolist() for i in range(qo.numel() - 1)]
    for policy, k in ((K.POLICY_LPM, 1), (K.POLICY_KLPM, 3), (K.POLICY_FCFS, 1)):
        got = run_gpu(K, prefill, prompts, w.arrivals, policy, k, start=w.start_tick)
        want = run_oracle(prefill, prompts, w.arrivals, policy, k, start=w.start_tick)
        same(got, want)


def test_tree_too_small_for_the_queue(K):
    """The grouped loop needs no room in the tree: every output is still produced, the insertion at the end
    reports the capacity error, and the tree stays usable."""
    prompts = [[1, 2, 3, 4, 5, 6, 7, 8, 9, 10], [1, 2, 3, 9, 9, 9, 9, 9, 9, 9], [5] * 12] * 30
    arr = list(range(len(prompts)))
    qt, qo = W.to_csr(prompts)
    tree = K.rt_create(max_nodes=256, max_pool_tokens=20, max_clock=256)
    n = len(prompts)
    order = torch.full((n,), -1, dtype=torch.int32, device="cuda")
    unc = torch.full((n,), -1, dtype=torch.int32, device="cuda")
    ttft = torch.full((n,), -1, dtype=torch.int64, device="cuda")
    K.klpm_run(tree, dev(qt), dev(qo), dev(torch.tensor(arr, dtype=torch.int64)), K.make_params(K.POLICY_LPM, 1), order, unc, ttft)
    assert K.rt_sync_status(tree) == K.RT_ERR_CAPACITY
    assert K.klpm_run_path(tree) == K.RUN_PATH_GROUPED
    want = run_oracle([], prompts, arr, oracle.POLICY_LPM, 1)
    assert np.array_equal(order.cpu().numpy(), want[0]) and np.array_equal(unc.cpu().numpy(), want[1])
    assert np.array_equal(ttft.cpu().numpy(), want[2])
    m = torch.zeros(n, dtype=torch.int32, device="cuda")
    K.rt_match_batch(tree, dev(qt), dev(qo), m)           # the partly filled tree still answers
    assert int(m.max()) <= 12
    K.rt_destroy(tree)


@pytest.mark.parametrize("n", [37, 1500, 5000])
def test_loop_started_from_the_records_of_a_batched_match(K, n):
    """rt_match_batch_ex keeps, per query, where its match ended; klpm_run_ex started from those records gives the
    oracle's schedule and tree, like the call that matches the queries itself (batches below and above the size
    from which the match takes its queries bucketed by first token)."""
    prompts, arr = shared_prefix_queue(41, n, [(12, 3), (9, 4)], tail=9, vocab=5, max_gap=2)
    prefill, _ = shared_prefix_queue(42, 300, [(12, 3), (9, 4)], tail=4, vocab=5, max_gap=0)
    for policy, k in ((K.POLICY_KLPM, 3), (K.POLICY_LPM, 1)):
        want = run_oracle(prefill, prompts, arr, policy, k)
        same(run_gpu(K, prefill, prompts, arr, policy, k, from_match=True), want)
        same(run_gpu(K, prefill, prompts, arr, policy, k), want)


def test_match_records_are_refused_once_they_are_stale(K):
    prompts, arr = shared_prefix_queue(43, 600, [(10, 3)], tail=6, vocab=4, max_gap=1)
    qt, qo = W.to_csr(prompts)
    n = len(prompts)
    tree = K.rt_create(max_nodes=4 * n + 16, max_pool_tokens=2 * qt.numel() + 16 * n + 16, max_clock=2 * n + 16)
    d_qt, d_qo, d_arr = dev(qt), dev(qo), dev(torch.as_tensor(arr, dtype=torch.int64))
    out = [torch.zeros(n, dtype=torch.int32, device="cuda"), torch.zeros(n, dtype=torch.int32, device="cuda"),
           torch.zeros(n, dtype=torch.int64, device="cuda")]
    state = K.match_state_buffer(n, "cuda")
    m = torch.zeros(n, dtype=torch.int32, device="cuda")
    p = K.make_params(K.POLICY_KLPM, 2)
    K.rt_match_batch_ex(tree, d_qt, d_qo, m, None, None, state)
    K.rt_insert(tree, d_qt, d_qo[:3])                      # the tree changes: the records no longer describe it
    with pytest.raises(K.KlpmError) as e:
        K.klpm_run_ex(tree, d_qt, d_qo, d_arr, p, None, 0, *out, None, state)
    assert e.value.code == K.RT_ERR_INVALID
    K.rt_match_batch_ex(tree, d_qt, d_qo, m, None, None, state)
    with pytest.raises(K.KlpmError):                        # another buffer than the one the match wrote
        K.klpm_run_ex(tree, d_qt, d_qo, d_arr, p, None, 0, *out, None, K.match_state_buffer(n, "cuda"))
    state.zero_()                                           # the caller overwrote the records: caught on the device
    K.klpm_run_ex(tree, d_qt, d_qo, d_arr, p, None, 0, *out, None, state)
    assert K.rt_sync_status(tree) == K.RT_ERR_INVALID and K.rt_status_detail(tree) == 110
    K.rt_destroy(tree)


def test_queue_above_the_shared_memory_bitmaps(K):
    """300,000 queries, everybody waiting: list mode with 64-slot leaf blocks and two of its bitmaps in global memory.
    The oracle's O(n^2) schedule is out of reach at this size, so the loop is compared bit for bit with the
    one-decision-at-a-time loop (which the oracle checks at the smaller sizes) and through what holds at any size."""
    n = 300_000
    rng = np.random.RandomState(5)
    heads = rng.randint(0, 50000, size=(64, 24))
    which = rng.randint(0, 64, size=n)
    cut = rng.randint(1, 25, size=n)
    tails = rng.randint(0, 50000, size=(n, 6))
    lens = cut + rng.randint(1, 7, size=n)
    off = np.zeros(n + 1, dtype=np.int64)
    off[1:] = np.cumsum(lens)
    tok = np.empty(off[-1], dtype=np.int32)
    for i in range(n):
        tok[off[i]:off[i] + cut[i]] = heads[which[i], :cut[i]]
        tok[off[i] + cut[i]:off[i + 1]] = tails[i, :lens[i] - cut[i]]
    arr = np.sort(rng.randint(0, 1000, size=n)).astype(np.int64)
    d_tok, d_off, d_arr = torch.from_numpy(tok).cuda(), torch.from_numpy(off).cuda(), torch.from_numpy(arr).cuda()
    outs = []
    for legacy in (False, True):
        tree = K.rt_create(max_nodes=2 * n + 64, max_pool_tokens=int(off[-1]) + 8 * n + 64, max_clock=n + 64)
        order = torch.full((n,), -1, dtype=torch.int32, device="cuda")
        unc = torch.full((n,), -1, dtype=torch.int32, device="cuda")
        ttft = torch.full((n,), -1, dtype=torch.int64, device="cuda")
        K.klpm_debug_set("run_one_by_one", 1 if legacy else 0)
        try:
            K.klpm_run(tree, d_tok, d_off, d_arr, K.make_params(K.POLICY_KLPM, 3, 0, 1, 1000), order, unc, ttft)
            assert K.rt_sync_status(tree) == 0
        finally:
            K.klpm_debug_set("run_one_by_one", -1)
        assert K.klpm_run_path(tree) == (K.RUN_PATH_ONE_BY_ONE if legacy else K.RUN_PATH_GROUPED)
        if not legacy:
            cn = K.rt_debug_counters(tree)
            assert cn["cta_batch_decisions"] + cn["warp_step_decisions"] + cn["single_decisions"] > n // 2      # list mode ran
        st = K.rt_stats(tree)
        outs.append((order.cpu().numpy(), unc.cpu().numpy(), ttft.cpu().numpy(), st))
        K.rt_destroy(tree)
    for a, b in zip(outs[0][:3], outs[1][:3]):
        assert np.array_equal(a, b)
    assert {f: outs[0][3][f] for f in ("n_nodes", "tokens", "clock")} == {f: outs[1][3][f] for f in ("n_nodes", "tokens", "clock")}
    order, unc = outs[0][0].astype(np.int64), outs[0][1].astype(np.int64)
    assert np.array_equal(np.sort(order), np.arange(n))
    assert int(unc.sum()) == outs[0][3]["tokens"]


@pytest.mark.parametrize("k", [2, 3, 4, 7, 40])
def test_long_batches_where_the_two_pick_orders_meet(K, k):
    """20,000 queries, everybody waiting, nobody grouped (every query ends its match with a token of its own), match
    lengths unrelated to the arrival order: CTA-wide batches run long and the oldest-first picks keep meeting
    list entries inside them -- once per batch (resolved inside the batch), several times (the batch ends before
    the second), with the two decisions close together and far apart.  Compared with the oracle's schedule."""
    n, trunks, depth = 20_000, 200, 60
    rng = np.random.RandomState(900 + k)
    trunk = rng.randint(0, 50000, size=(trunks, depth))
    prefill = [trunk[r].tolist() for r in range(trunks)]
    prompts = []
    for i in range(n):
        r, p = rng.randint(trunks), rng.randint(1, depth)
        prompts.append(trunk[r, :p].tolist() + [50000 + i] + rng.randint(0, 50000, size=rng.randint(0, 3)).tolist())
    arr = [0] * n
    got = run_gpu(K, prefill, prompts, arr, 2, k)
    want = run_oracle(prefill, prompts, arr, 2, k)
    same(got, want)
