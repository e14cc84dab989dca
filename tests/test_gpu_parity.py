"""CUDA path vs CPU oracle, element by element, through the C ABI.  Integer work: the bar is bit-exact."""
import numpy as np
import pytest
import torch

import oracle
from oracle import definition as D
from paper_2502_04677_b200 import workloads as W

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def K():
    from paper_2502_04677_b200 import binding
    return binding


def dev(t):
    return t.cuda() if isinstance(t, torch.Tensor) else torch.as_tensor(t).cuda()


def csr(prompts):
    return W.to_csr(prompts)


def caps(*token_counts, n_prompts=0):
    total = int(sum(token_counts))
    return dict(max_nodes=2 * n_prompts + 16, max_pool_tokens=total + 8 * n_prompts + 16, max_clock=n_prompts + 16)


def gpu_tree(K, tokens, offsets, extra_prompts=0, extra_tokens=0, budget=0):
    n = offsets.numel() - 1
    c = caps(tokens.numel(), extra_tokens, n_prompts=n + extra_prompts)
    if n == 0:
        return K.rt_create(budget_tokens=budget, **c)
    return K.rt_build(dev(tokens), dev(offsets), budget_tokens=budget, **c)


def gpu_match(K, tree, qt, qo):
    nq = qo.numel() - 1
    m = torch.full((nq,), -7, dtype=torch.int32, device="cuda")
    node = torch.full((nq,), -7, dtype=torch.int32, device="cuda")
    off = torch.full((nq,), -7, dtype=torch.int32, device="cuda")
    K.rt_match_batch(tree, dev(qt), dev(qo), m, node, off)
    assert K.rt_sync_status(tree) == 0
    return m.cpu().numpy(), node.cpu().numpy(), off.cpu().numpy()


def oracle_tree(tokens, offsets, budget=0):
    t = oracle.OracleTree(budget)
    if offsets.numel() > 1:
        t.insert(tokens.numpy(), offsets.numpy())
    return t


# ------------------------------------------------------------------ batched match

def assert_match_equals_oracle(K, tree, ot, qt, qo):
    """Match length and where the match ended (tokens matched of the edge holding the last matched token; the
    depth at which that edge starts is the difference), element by element."""
    m, node, off = gpu_match(K, tree, qt, qo)
    want_m, want_off, want_depth = ot.match_pos(qt.numpy(), qo.numpy())
    assert np.array_equal(m, want_m)
    assert np.array_equal(off, want_off)
    assert np.array_equal(m - off, want_depth)
    assert np.array_equal(node == 0, m == 0)
    return m


def check_match(K, pt, po, qt, qo):
    tree = gpu_tree(K, pt, po)
    ot = oracle_tree(pt, po)
    m = assert_match_equals_oracle(K, tree, ot, qt, qo)
    st, ost = K.rt_stats(tree), ot.stats()
    assert (st["n_nodes"], st["tokens"], st["clock"]) == (ost["n_nodes"], ost["tokens"], ost["clock"])
    K.rt_destroy(tree)
    return m


def test_match_tiny_config(K):
    w = W.tiny()
    pt, po = w.prefill.materialize()
    qt, qo = w.queries.materialize()
    m = check_match(K, pt, po, qt, qo)
    assert m.min() >= 512          # every query shares one of the 8 cached prefixes


@pytest.mark.parametrize("seed", range(4))
def test_match_small_alphabet_ragged_and_empty(K, seed):
    """Frequent overlaps, empty prompts and queries, lengths that straddle the 128-token compare chunk."""
    cached, _ = W.random_small_queue(seed, 300, vocab=2, max_len=400)
    queries, _ = W.random_small_queue(seed + 50, 257, vocab=2, max_len=420)
    long_a = [1] * 1000 + [0]
    cached += [long_a, [1] * 127, [1] * 128 + [0], [0] * 129, []]
    queries += [[1] * 1000, [1] * 1001, long_a + [1], [1] * 128, [0] * 130, [], [1] * 127 + [0]]
    check_match(K, *csr(cached), *csr(queries))
    # brute force against every cached prompt as well (definition of the match length)
    tree = gpu_tree(K, *csr(cached))
    m, _, _ = gpu_match(K, tree, *csr(queries))
    ct, co = csr(cached)
    qt, qo = csr(queries)
    assert np.array_equal(m, oracle.match_bruteforce(qt.numpy(), qo.numpy(), ct.numpy(), co.numpy()))


def test_match_empty_tree_and_no_queries(K):
    tree = K.rt_create(max_nodes=16, max_pool_tokens=16)
    qt, qo = csr([[1, 2, 3], []])
    m, node, off = gpu_match(K, tree, qt, qo)
    assert m.tolist() == [0, 0] and node.tolist() == [0, 0]
    K.rt_match_batch(tree, dev(qt), dev(torch.zeros(1, dtype=torch.int64)), torch.empty(0, dtype=torch.int32, device="cuda"))
    assert K.rt_sync_status(tree) == 0


@pytest.mark.parametrize("name,scale", [("medium", 1 / 64), ("hierarchical", 1 / 512), ("adversarial", 1 / 1024)])
def test_match_scaled_configs(K, name, scale):
    w = W.WORKLOADS[name](scale=scale)
    pt, po = w.prefill.materialize()
    qt, qo = w.queries.materialize()
    check_match(K, pt, po, qt, qo)


# ------------------------------------------------------------------ insert

@pytest.mark.parametrize("budget", [0, 60])
def test_insert_new_tokens_and_stats(K, budget):
    prompts, _ = W.random_small_queue(9, 200, vocab=2, max_len=16, min_len=0)
    pt, po = csr(prompts)
    tree = K.rt_create(budget_tokens=budget, **caps(pt.numel(), n_prompts=len(prompts)))
    new = torch.zeros(len(prompts), dtype=torch.int32, device="cuda")
    half = len(prompts) // 2
    K.rt_insert(tree, dev(pt), dev(po[:half + 1]), new[:half])
    K.rt_insert(tree, dev(pt), dev(po[half:]), new[half:])
    assert K.rt_sync_status(tree) == 0
    ot = oracle.OracleTree(budget)
    want = ot.insert(pt.numpy(), po.numpy())
    assert np.array_equal(new.cpu().numpy(), want)
    st, ost = K.rt_stats(tree), ot.stats()
    for key in ("n_nodes", "tokens", "clock", "evictions"):
        assert st[key] == ost[key], key
    if budget:
        assert ost["evictions"] > 0 and st["tokens"] <= budget
    qs, _ = W.random_small_queue(10, 100, vocab=2, max_len=18)
    assert_match_equals_oracle(K, tree, ot, *csr(qs))        # hop-by-hop walk on a tree with a budget too


def test_capacity_and_budget_errors_are_reported_not_fatal(K):
    pt, po = csr([[1, 2, 3, 4, 5, 6, 7, 8], [9, 9, 9]])
    tree = K.rt_create(max_nodes=64, max_pool_tokens=4)
    K.rt_insert(tree, dev(pt), dev(po))
    assert K.rt_sync_status(tree) == K.RT_ERR_CAPACITY
    tree2 = K.rt_create(max_nodes=64, max_pool_tokens=64, budget_tokens=5)
    K.rt_insert(tree2, dev(pt), dev(po))
    assert K.rt_sync_status(tree2) == K.RT_ERR_BUDGET
    # the device is still usable
    tree3 = K.rt_build(dev(pt), dev(po), max_nodes=64, max_pool_tokens=64)
    m, _, _ = gpu_match(K, tree3, *csr([[1, 2, 3, 9]]))
    assert m.tolist() == [3]


def test_invalid_arguments(K):
    with pytest.raises(K.KlpmError) as e:
        K.rt_create(max_nodes=0, max_pool_tokens=10)
    assert e.value.code == K.RT_ERR_INVALID
    tree = K.rt_create(max_nodes=16, max_pool_tokens=16)
    z = torch.zeros(4, dtype=torch.int32, device="cuda")
    a = torch.zeros(4, dtype=torch.int64, device="cuda")
    wmask = torch.ones(4, dtype=torch.uint8, device="cuda")
    pick = torch.zeros(1, dtype=torch.int32, device="cuda")
    with pytest.raises(K.KlpmError):
        K.klpm_select(z, a, wmask, 0, K.make_params(K.POLICY_KLPM, k=0), pick)
    with pytest.raises(K.KlpmError):
        K.klpm_select(z, a, wmask, -1, K.make_params(K.POLICY_KLPM, k=2), pick)
    with pytest.raises(ValueError):
        K.rt_match_batch(tree, torch.zeros(4, dtype=torch.int32), a, z)     # CPU tensor: no CPU path


# ------------------------------------------------------------------ selection (one decision)


@pytest.mark.parametrize("n", [1, 33, 1000, 70001])
def test_select_single_decision(K, n):
    g = torch.Generator().manual_seed(n)
    m = torch.randint(0, 6, (n,), generator=g, dtype=torch.int32)
    t = torch.randint(0, 50, (n,), generator=g, dtype=torch.int64) * (1 << 33)
    waiting = (torch.rand(n, generator=g) < 0.7).to(torch.uint8)
    pick = torch.zeros(1, dtype=torch.int32, device="cuda")
    for policy, k, c in [(0, 1, 0), (1, 1, 5), (2, 3, 0), (2, 3, 1), (2, 3, 2), (2, 3, 3), (2, 1, 7)]:
        K.klpm_select(dev(m), dev(t), dev(waiting), c, K.make_params(policy, k), pick)
        assert int(pick.item()) == oracle.select(m.numpy(), t.numpy(), waiting.numpy(), c, policy, k)
    K.klpm_select(dev(m), dev(t), dev(torch.zeros(n, dtype=torch.uint8)), 1, K.make_params(1), pick)
    assert int(pick.item()) == -1


# ------------------------------------------------------------------ replay along a fixed order

@pytest.mark.parametrize("budget", [0, 50])
def test_replay_fixed_order(K, budget):
    prompts, arr = W.random_small_queue(21, 150, vocab=2, max_len=16, min_len=1, max_gap=9)
    prefill, _ = W.random_small_queue(22, 20, vocab=2, max_len=12, min_len=1)
    qt, qo = csr(prompts)
    pt, po = csr(prefill)
    order = torch.randperm(len(prompts), generator=torch.Generator().manual_seed(1)).to(torch.int32)
    tree = gpu_tree(K, pt, po, extra_prompts=len(prompts), extra_tokens=qt.numel(), budget=budget)
    n = len(prompts)
    unc = torch.full((n,), -1, dtype=torch.int32, device="cuda")
    ttft = torch.full((n,), -1, dtype=torch.int64, device="cuda")
    comp = torch.full((n,), -1, dtype=torch.int64, device="cuda")
    p = K.make_params(K.POLICY_FCFS, 1, c_num=1, c_den=3, start_tick=5)
    K.klpm_replay(tree, dev(order), dev(qt), dev(qo), dev(torch.tensor(arr)), p, unc, ttft, comp)
    assert K.rt_sync_status(tree) == 0
    ot = oracle_tree(pt, po, budget)
    ou, ottft, ocomp = oracle.replay(order.numpy(), qt.numpy(), qo.numpy(), arr, 1, 3, 5, oracle.CACHE_TREE, ot)
    assert np.array_equal(unc.cpu().numpy(), ou)
    assert np.array_equal(ttft.cpu().numpy(), ottft)
    assert np.array_equal(comp.cpu().numpy(), ocomp)
    assert K.rt_stats(tree)["evictions"] == ot.stats()["evictions"]


@pytest.mark.parametrize("budget", [0, 4000])
def test_replay_both_forms_on_a_longer_queue(K, budget):
    """6,000 prompts with shared blocks, a random order of 4,500 of them, c_attn = 1/2: the replay through the device
    loop, the plain one-prompt-after-the-other form (debug setting) and the oracle agree on every output and on the
    tree that is left (match of every prompt afterwards)."""
    rng = np.random.RandomState(3)
    blocks = [rng.randint(0, 6, size=10).tolist() for _ in range(5)]
    prompts = [blocks[rng.randint(5)] + blocks[rng.randint(5)][:rng.randint(1, 11)] + rng.randint(0, 6, size=rng.randint(0, 7)).tolist()
               for _ in range(6000)]
    arr = np.cumsum(rng.randint(0, 3, size=6000)).tolist()
    qt, qo = csr(prompts)
    order = torch.from_numpy(rng.permutation(6000)[:4500].astype(np.int32))
    n = len(prompts)
    got = []
    for plain in (False, True):
        tree = K.rt_create(budget_tokens=budget, **caps(qt.numel(), n_prompts=n))
        unc = torch.full((n,), -1, dtype=torch.int32, device="cuda")
        ttft = torch.full((n,), -1, dtype=torch.int64, device="cuda")
        comp = torch.full((n,), -1, dtype=torch.int64, device="cuda")
        K.klpm_debug_set("run_one_by_one", 1 if plain else 0)
        try:
            K.klpm_replay(tree, dev(order), dev(qt), dev(qo), dev(torch.tensor(arr)), K.make_params(K.POLICY_FCFS, 1, 1, 2, 3), unc, ttft, comp)
            assert K.rt_sync_status(tree) == 0
        finally:
            K.klpm_debug_set("run_one_by_one", -1)
        m, _, off = gpu_match(K, tree, qt, qo)
        got.append((unc.cpu().numpy(), ttft.cpu().numpy(), comp.cpu().numpy(), m, off, K.rt_stats(tree)))
        K.rt_destroy(tree)
    ot = oracle.OracleTree(budget)
    ou, ottft, ocomp = oracle.replay(order.numpy(), qt.numpy(), qo.numpy(), arr, 1, 2, 3, oracle.CACHE_TREE, ot)
    want_u, want_t, want_c = (np.full(n, -1, dtype=x.dtype) for x in (ou, ottft, ocomp))
    idx = order.numpy()
    want_u[idx], want_t[idx], want_c[idx] = ou[idx], ottft[idx], ocomp[idx]
    om, ooff, _ = ot.match_pos(qt.numpy(), qo.numpy())
    for g in got:
        assert np.array_equal(g[0], want_u) and np.array_equal(g[1], want_t) and np.array_equal(g[2], want_c)
        assert np.array_equal(g[3], om) and np.array_equal(g[4], ooff)
        for key in ("n_nodes", "tokens", "clock", "evictions"):
            assert g[5][key] == ot.stats()[key], key
    if budget:
        assert ot.stats()["evictions"] > 0


def test_replay_stops_at_an_order_entry_that_is_not_a_query(K):
    """An order with -1 (or an index past the queue) in it: the replay processes what comes before, touches nothing
    for the bad entry or after it, and reports RT_ERR_INVALID through the status word."""
    prompts, arr = W.random_small_queue(23, 12, vocab=3, max_len=9, min_len=1)
    qt, qo = csr(prompts)
    n = len(prompts)
    for bad in (-1, n, 1 << 30, 3):                       # not a query, or a query that was processed already
        tree = K.rt_create(**caps(qt.numel(), n_prompts=n))
        order = torch.tensor([3, 1, bad, 2], dtype=torch.int32)
        unc = torch.full((n,), -1, dtype=torch.int32, device="cuda")
        ttft = torch.full((n,), -1, dtype=torch.int64, device="cuda")
        K.klpm_replay(tree, dev(order), dev(qt), dev(qo), dev(torch.tensor(arr)), K.make_params(K.POLICY_FCFS), unc, ttft)
        assert K.rt_sync_status(tree) == K.RT_ERR_INVALID and K.rt_status_detail(tree) == 108
        ou, ottft, _ = oracle.replay([3, 1], qt.numpy(), qo.numpy(), arr, cache_mode=oracle.CACHE_TREE)
        want_u = np.full(n, -1, dtype=np.int32)
        want_t = np.full(n, -1, dtype=np.int64)
        want_u[[3, 1]] = ou[[3, 1]]
        want_t[[3, 1]] = ottft[[3, 1]]
        assert np.array_equal(unc.cpu().numpy(), want_u) and np.array_equal(ttft.cpu().numpy(), want_t)
        assert K.rt_stats(tree)["clock"] == 2
        K.rt_destroy(tree)


# ------------------------------------------------------------------ the whole loop

def run_gpu(K, pt, po, qt, qo, arr, policy, k, budget=0, start=0, c_num=0, c_den=1):
    n = qo.numel() - 1
    tree = gpu_tree(K, pt, po, extra_prompts=n, extra_tokens=qt.numel(), budget=budget)
    order = torch.full((n,), -1, dtype=torch.int32, device="cuda")
    unc = torch.full((n,), -1, dtype=torch.int32, device="cuda")
    ttft = torch.full((n,), -1, dtype=torch.int64, device="cuda")
    comp = torch.full((n,), -1, dtype=torch.int64, device="cuda")
    K.klpm_run(tree, dev(qt), dev(qo), dev(torch.as_tensor(arr, dtype=torch.int64)),
               K.make_params(policy, k, c_num, c_den, start), order, unc, ttft, comp)
    assert K.rt_sync_status(tree) == 0
    st = K.rt_stats(tree)
    K.rt_destroy(tree)
    return order.cpu().numpy(), unc.cpu().numpy(), ttft.cpu().numpy(), comp.cpu().numpy(), st


def run_oracle(pt, po, qt, qo, arr, policy, k, budget=0, start=0, c_num=0, c_den=1, tier=oracle.TIER_UPDATE):
    ot = oracle_tree(pt, po, budget)
    out = oracle.schedule(qt.numpy(), qo.numpy(), np.asarray(arr, dtype=np.int64), policy, k, c_num, c_den, start,
                          oracle.CACHE_TREE, tier, ot)
    return out + (ot.stats(),)


def assert_same_schedule(got, want):
    for g, w, name in zip(got[:4], want[:4], ("order", "uncached", "ttft", "completion")):
        assert np.array_equal(g, w), name
    for key in ("n_nodes", "tokens", "clock", "evictions"):
        assert got[4][key] == want[4][key], key


def test_run_toy_example_on_device(K):
    """Section 4.2's toy example with the whole tree cached: LPM / 2-LPM order x1,x3,x2,x4, TTFT 10,15,25,30."""
    prompts, arr = W.regular_arrival_shuffled_queue(4, 2, 5, 5, 0, [1, 2, 3, 4])
    qt, qo = csr(prompts)
    e = torch.zeros(0, dtype=torch.int32), torch.zeros(1, dtype=torch.int64)
    for policy, k in ((K.POLICY_LPM, 1), (K.POLICY_KLPM, 2)):
        order, unc, ttft, comp, _ = run_gpu(K, *e, qt, qo, arr, policy, k)
        assert order.tolist() == [0, 2, 1, 3] and ttft.tolist() == [10, 25, 15, 30]
    order, unc, ttft, comp, _ = run_gpu(K, *e, qt, qo, arr, K.POLICY_FCFS, 1)
    assert order.tolist() == [0, 1, 2, 3] and ttft.tolist() == [10, 20, 25, 30]


@pytest.mark.parametrize("seed", range(6))
@pytest.mark.parametrize("budget", [0, 48])
def test_run_fuzz_small_alphabet(K, seed, budget):
    """Tiny alphabet: ties, identical prompts, prompts that are prefixes of others, idle periods, eviction."""
    prompts, arr = W.random_small_queue(seed + 700, 120, vocab=2, max_len=14, min_len=0, max_gap=5)
    prefill, _ = W.random_small_queue(seed + 800, 12, vocab=2, max_len=10, min_len=1)
    qt, qo = csr(prompts)
    pt, po = csr(prefill)
    for policy, k in ((0, 1), (1, 1), (2, 1), (2, 2), (2, 3), (2, 200)):
        got = run_gpu(K, pt, po, qt, qo, arr, policy, k, budget=budget, c_num=1, c_den=2)
        want = run_oracle(pt, po, qt, qo, arr, policy, k, budget=budget, c_num=1, c_den=2, tier=oracle.TIER_REMATCH)
        assert_same_schedule(got, want)
        ref = D.schedule(prompts, arr, policy, k, 1, 2, 0, D.TREE, prefill, budget)
        assert got[0].tolist() == ref[0] and got[2].tolist() == ref[2]


def test_run_tiny_config_full(K):
    """Configuration 'tiny' as stated: 1,000 waiting queries, tree of 2,000 prompts, k = 2; oracle re-matches every pick."""
    w = W.tiny()
    pt, po = w.prefill.materialize()
    qt, qo = w.queries.materialize()
    got = run_gpu(K, pt, po, qt, qo, w.arrivals, K.POLICY_KLPM, 2, start=w.start_tick)
    want = run_oracle(pt, po, qt, qo, w.arrivals, oracle.POLICY_KLPM, 2, start=w.start_tick, tier=oracle.TIER_REMATCH)
    assert_same_schedule(got, want)
    # unbounded tree cache: total uncached tokens = growth of the tree
    assert int(got[1].sum()) == got[4]["tokens"] - int(oracle_tree(pt, po).stats()["tokens"])


@pytest.mark.parametrize("k", [1, 2, 4, 8])
def test_run_medium_scaled(K, k):
    w = W.medium(scale=1 / 32)
    pt, po = w.prefill.materialize()
    qt, qo = w.queries.materialize()
    got = run_gpu(K, pt, po, qt, qo, w.arrivals, K.POLICY_KLPM, k, start=w.start_tick)
    want = run_oracle(pt, po, qt, qo, w.arrivals, oracle.POLICY_KLPM, k, start=w.start_tick)
    assert_same_schedule(got, want)


@pytest.mark.parametrize("policy,k", [(0, 1), (1, 1), (2, 4)])
def test_run_streaming_scaled_with_lru(K, policy, k):
    """Poisson arrivals from an empty tree under a KV budget with LRU eviction; per-query integer TTFT."""
    w = W.streaming(scale=1 / 100)
    qt, qo = w.queries.materialize()
    e = torch.zeros(0, dtype=torch.int32), torch.zeros(1, dtype=torch.int64)
    got = run_gpu(K, *e, qt, qo, w.arrivals, policy, k, budget=w.budget_tokens)
    want = run_oracle(*e, qt, qo, w.arrivals, policy, k, budget=w.budget_tokens)
    assert_same_schedule(got, want)
    assert want[4]["evictions"] > 0


@pytest.mark.parametrize("name,scale,k", [("hierarchical", 1 / 256, 4), ("adversarial", 1 / 512, 4)])
def test_run_scaled_configs(K, name, scale, k):
    w = W.WORKLOADS[name](scale=scale)
    pt, po = w.prefill.materialize()
    qt, qo = w.queries.materialize()
    got = run_gpu(K, pt, po, qt, qo, w.arrivals, K.POLICY_KLPM, k, start=w.start_tick)
    want = run_oracle(pt, po, qt, qo, w.arrivals, oracle.POLICY_KLPM, k, start=w.start_tick)
    assert_same_schedule(got, want)


# ------------------------------------------------------------------ bulk insertion, checkpoint / rollback

@pytest.mark.parametrize("seed", range(3))
def test_bulk_insert_equals_sequential_insert(K, seed):
    """Concurrent insertion in rounds gives the same cached prefixes and node boundaries as one-by-one."""
    prompts, _ = W.random_small_queue(seed + 900, 700, vocab=2, max_len=40, min_len=0)
    prompts += [[1] * 300, [1] * 300, [1] * 150, [1] * 299 + [0], []]
    pt, po = csr(prompts)
    c = caps(pt.numel(), n_prompts=len(prompts))
    bulk = K.rt_build(dev(pt), dev(po), **c)                       # n >= 64, no budget: rounds
    seq = K.rt_create(**c)
    new = torch.zeros(len(prompts), dtype=torch.int32, device="cuda")
    K.rt_insert(seq, dev(pt), dev(po), new)                        # asks for new_tokens: one by one
    assert K.rt_sync_status(bulk) == 0 and K.rt_sync_status(seq) == 0
    a, b = K.rt_stats(bulk), K.rt_stats(seq)
    ost = oracle_tree(pt, po).stats()
    for key in ("n_nodes", "tokens", "clock"):
        assert a[key] == b[key] == ost[key], key
    qs, _ = W.random_small_queue(seed + 950, 300, vocab=2, max_len=45)
    qt, qo = csr(qs)
    ma, _, _ = gpu_match(K, bulk, qt, qo)
    mb, _, _ = gpu_match(K, seq, qt, qo)
    assert np.array_equal(ma, mb)
    # a second bulk batch on top of the first
    more, _ = W.random_small_queue(seed + 960, 200, vocab=2, max_len=40, min_len=1)
    mt, mo = csr(more)
    big = K.rt_build(dev(pt), dev(po), **caps(pt.numel(), mt.numel(), n_prompts=len(prompts) + len(more)))
    K.rt_insert(big, dev(mt), dev(mo))
    ot = oracle_tree(pt, po)
    ot.insert(mt.numpy(), mo.numpy())
    st = K.rt_stats(big)
    assert (st["n_nodes"], st["tokens"], st["clock"]) == (ot.stats()["n_nodes"], ot.stats()["tokens"], ot.stats()["clock"])
    m, _, _ = gpu_match(K, big, qt, qo)
    assert np.array_equal(m, ot.match(qt.numpy(), qo.numpy()))


def test_checkpoint_and_rollback(K):
    w = W.medium(scale=1 / 128)
    pt, po = w.prefill.materialize()
    qt, qo = w.queries.materialize()
    n = qo.numel() - 1
    tree = gpu_tree(K, pt, po, extra_prompts=2 * n, extra_tokens=2 * qt.numel())
    K.rt_checkpoint(tree)
    before = K.rt_stats(tree)
    outs = []
    for _ in range(2):
        order = torch.zeros(n, dtype=torch.int32, device="cuda")
        unc = torch.zeros(n, dtype=torch.int32, device="cuda")
        ttft = torch.zeros(n, dtype=torch.int64, device="cuda")
        K.klpm_run(tree, dev(qt), dev(qo), dev(w.arrivals), K.make_params(K.POLICY_KLPM, 4, start_tick=w.start_tick),
                   order, unc, ttft)
        assert K.rt_sync_status(tree) == 0
        assert K.rt_stats(tree)["tokens"] > before["tokens"]
        outs.append((order.cpu(), unc.cpu(), ttft.cpu()))
        K.rt_rollback(tree)
        after = K.rt_stats(tree)
        assert {k: after[k] for k in ("n_nodes", "tokens", "clock")} == {k: before[k] for k in ("n_nodes", "tokens", "clock")}
    for a, b in zip(outs[0], outs[1]):
        assert torch.equal(a, b)
    m, _, _ = gpu_match(K, tree, qt, qo)
    assert np.array_equal(m, oracle_tree(pt, po).match(qt.numpy(), qo.numpy()))


# ------------------------------------------------------------------ prefix-to-prompt ratio experiment (Appendix C.2)

@pytest.mark.parametrize("u,d", [(1000, 5000), (3000, 3000), (5000, 1000)])
def test_run_prefix_ratio_experiment(K, u, d):
    """n = 2000 random-string prompts, 4 replicas per prefix, Poisson 80/s, policies k = 1, 4 and LPM."""
    w = W.prefix_ratio(u, d)
    qt, qo = w.queries.materialize()
    e = torch.zeros(0, dtype=torch.int32), torch.zeros(1, dtype=torch.int64)
    for policy, k in ((K.POLICY_KLPM, 1), (K.POLICY_KLPM, 4), (K.POLICY_LPM, 1)):
        got = run_gpu(K, *e, qt, qo, w.arrivals, policy, k)
        want = run_oracle(*e, qt, qo, w.arrivals, policy, k)
        assert_same_schedule(got, want)
    # every prefix is prefilled once, every doc once: total uncached tokens under an unbounded tree cache
    assert int(got[1].sum()) == (w.queries.n // 4) * u + w.queries.n * d


# ------------------------------------------------------------------ long edges, every alignment, degenerate streams

def test_match_long_edges_all_alignments(K):
    """One 70,001-token cached prompt plus prefixes of it; queries that agree with it for every length in a
    ragged set (around the 128-token chunks and the 16-byte units), starting at every 4-byte phase."""
    g = torch.Generator().manual_seed(7)
    base = torch.randint(0, 50000, (70001,), generator=g, dtype=torch.int32).tolist()
    cached = [base, base[:4097], base[:130] + [7, 7, 7], base[:1]]
    lens = [0, 1, 2, 3, 4, 5, 127, 128, 129, 255, 256, 257, 511, 4096, 4097, 4098, 65535, 70000, 70001]
    queries = []
    for i, n in enumerate(lens):
        queries.append(base[:n] + [60000 + i])            # diverges right after n tokens
        queries.append(base[:n])                          # ends there
        queries.append([1] * (i % 4))                     # filler that shifts the alignment of what follows
    check_match(K, *csr(cached), *csr(queries))


def test_run_degenerate_streams(K):
    e = torch.zeros(0, dtype=torch.int32), torch.zeros(1, dtype=torch.int64)
    # one query; identical prompts arriving together; empty prompts; everything at the same tick
    for prompts, arr in [([[5, 6, 7]], [3]),
                         ([[1, 2, 3]] * 9, [0] * 9),
                         ([[], [], [4], []], [0, 0, 0, 0]),
                         ([[9] * 300, [9] * 299 + [1], [9] * 300 + [2], [9] * 150], [5, 5, 5, 5])]:
        qt, qo = csr(prompts)
        for policy, k in ((0, 1), (1, 1), (2, 2)):
            got = run_gpu(K, *e, qt, qo, arr, policy, k)
            want = run_oracle(*e, qt, qo, arr, policy, k, tier=oracle.TIER_REMATCH)
            assert_same_schedule(got, want)


@pytest.mark.parametrize("n,kk", [(1, 3), (50, 7), (5000, 1), (5000, 16), (300001, 64)])
def test_select_topk_snapshot(K, n, kk):
    g = torch.Generator().manual_seed(n + kk)
    m = torch.randint(0, 4, (n,), generator=g, dtype=torch.int32)
    t = torch.randint(0, 30, (n,), generator=g, dtype=torch.int64) * (1 << 35)
    waiting = (torch.rand(n, generator=g) < 0.5).to(torch.uint8)
    out = torch.full((kk,), -9, dtype=torch.int32, device="cuda")
    for _ in range(2):                                   # the scratch is reused
        K.klpm_select_topk(dev(m), dev(t), dev(waiting), out)
        left, want = waiting.numpy().copy(), []           # the oracle's longest-match pick, kk times over what is left
        for _j in range(kk):
            want.append(oracle.select(m.numpy(), t.numpy(), left, 1, oracle.POLICY_LPM))
            if want[-1] >= 0:
                left[want[-1]] = 0
        assert out.tolist() == want
    # its first entry is klpm_select's longest-match pick
    pick = torch.zeros(1, dtype=torch.int32, device="cuda")
    K.klpm_select(dev(m), dev(t), dev(waiting), 1, K.make_params(K.POLICY_LPM), pick)
    assert int(pick.item()) == want[0]


@pytest.mark.parametrize("B", [1, 2, 7, 64, 100000])
def test_batch_times(K, B):
    w = W.medium(scale=1 / 64)
    pt, po = w.prefill.materialize()
    qt, qo = w.queries.materialize()
    order, unc, ttft, comp, _ = run_gpu(K, pt, po, qt, qo, w.arrivals, K.POLICY_KLPM, 4, start=w.start_tick)
    n = len(order)
    tb = torch.full((n,), -1, dtype=torch.int64, device="cuda")
    cb = torch.full((n,), -1, dtype=torch.int64, device="cuda")
    K.klpm_batch_times(dev(torch.from_numpy(order)), dev(w.arrivals), dev(torch.from_numpy(comp)), B, tb, cb)
    ot, oc = oracle.batch_times(order, w.arrivals.numpy(), comp, B)
    assert np.array_equal(tb.cpu().numpy(), ot) and np.array_equal(cb.cpu().numpy(), oc)


def test_batch_times_skips_order_entries_that_are_not_queries(K):
    order = torch.tensor([2, 0, -1, 1, 7, 3], dtype=torch.int32)      # 4 queries; bins of 2: (2,0) (-1,1) (7,3)
    arr = torch.tensor([0, 1, 2, 3], dtype=torch.int64)
    comp = torch.tensor([20, 40, 10, 60], dtype=torch.int64)
    tb = torch.full((4,), -1, dtype=torch.int64, device="cuda")
    cb = torch.full((4,), -1, dtype=torch.int64, device="cuda")
    skipped = torch.full((1,), -1, dtype=torch.int32, device="cuda")
    K.klpm_batch_times(dev(order), dev(arr), dev(comp), 2, tb, cb, skipped)
    # bin 1 finishes with query 0 (20); bin 2 with query 1 (40), its first entry is skipped; bin 3 with query 3 (60)
    assert cb.tolist() == [20, 40, 20, 60] and tb.tolist() == [20, 39, 18, 57]
    assert int(skipped.item()) == 2


# ------------------------------------------------------------------ queues large enough for the multi-CTA loop
# (above 4,096 queries klpm_run uses a sequencer CTA plus scanner CTAs and publishes picks early)

@pytest.mark.parametrize("k", [1, 3])
def test_run_multi_cta_all_waiting(K, k):
    w = W.medium(scale=1 / 4)
    assert w.queries.n > 4096
    pt, po = w.prefill.materialize()
    qt, qo = w.queries.materialize()
    got = run_gpu(K, pt, po, qt, qo, w.arrivals, K.POLICY_KLPM, k, start=w.start_tick)
    want = run_oracle(pt, po, qt, qo, w.arrivals, oracle.POLICY_KLPM, k, start=w.start_tick)
    assert_same_schedule(got, want)


@pytest.mark.parametrize("policy,k", [(2, 4), (1, 1)])
def test_run_multi_cta_streaming_with_lru(K, policy, k):
    w = W.streaming(scale=1 / 20)
    assert w.queries.n > 4096
    qt, qo = w.queries.materialize()
    e = torch.zeros(0, dtype=torch.int32), torch.zeros(1, dtype=torch.int64)
    got = run_gpu(K, *e, qt, qo, w.arrivals, policy, k, budget=w.budget_tokens)
    want = run_oracle(*e, qt, qo, w.arrivals, policy, k, budget=w.budget_tokens)
    assert_same_schedule(got, want)
    assert want[4]["evictions"] > 0


def test_run_multi_cta_ratio_experiment(K):
    w = W.prefix_ratio(3000, 3000, scale=2.5)          # 5,000 queries arriving over time, empty tree
    assert w.queries.n > 4096
    qt, qo = w.queries.materialize()
    e = torch.zeros(0, dtype=torch.int32), torch.zeros(1, dtype=torch.int64)
    for policy, k in ((K.POLICY_KLPM, 4), (K.POLICY_LPM, 1)):
        got = run_gpu(K, *e, qt, qo, w.arrivals, policy, k)
        want = run_oracle(*e, qt, qo, w.arrivals, policy, k)
        assert_same_schedule(got, want)


def test_match_after_the_loop_has_grown_the_tree(K):
    """The scheduling loop cuts edges and appends leaves; the batched match (which streams along contiguous
    pool runs) must see the grown tree exactly as the oracle's tree after the same schedule."""
    w = W.adversarial(scale=1 / 32)
    pt, po = w.prefill.materialize()
    qt, qo = w.queries.materialize()
    n = w.queries.n
    tree = gpu_tree(K, pt, po, extra_prompts=n, extra_tokens=qt.numel())
    order = torch.zeros(n, dtype=torch.int32, device="cuda")
    unc = torch.zeros(n, dtype=torch.int32, device="cuda")
    ttft = torch.zeros(n, dtype=torch.int64, device="cuda")
    half = 3 * n // 4                               # schedule the first part of the stream only
    assert half > 4096                              # large enough for the multi-CTA loop
    K.klpm_run(tree, dev(qt), dev(qo[:half + 1]), dev(w.arrivals[:half]), K.make_params(K.POLICY_KLPM, 4, 0, 1, w.start_tick),
               order[:half], unc[:half], ttft[:half])
    assert K.rt_sync_status(tree) == 0
    m, node, off = gpu_match(K, tree, qt, qo)
    ot = oracle_tree(pt, po)
    oracle.schedule(qt.numpy(), qo[:half + 1].numpy(), w.arrivals[:half].numpy(), oracle.POLICY_KLPM, 4, 0, 1, w.start_tick,
                    oracle.CACHE_TREE, oracle.TIER_UPDATE, ot)
    want = ot.match(qt.numpy(), qo.numpy())
    assert np.array_equal(m, want)
    lens = (qo[1:] - qo[:-1]).numpy()
    assert np.array_equal(m[:half], lens[:half])    # what was processed is fully cached
    st, ost = K.rt_stats(tree), ot.stats()
    assert (st["n_nodes"], st["tokens"], st["clock"]) == (ost["n_nodes"], ost["tokens"], ost["clock"])


def test_concurrent_k_sweep_on_clones(K):
    """Back-testing k: one stream of queries scheduled with k = 1, 2, 4, 8 at the same time, each on its own
    clone of the tree and its own CUDA stream.  Every run must equal the oracle's run for that k."""
    w = W.medium(scale=1 / 4)
    pt, po = w.prefill.materialize()
    qt, qo = w.queries.materialize()
    n = w.queries.n
    base = gpu_tree(K, pt, po, extra_prompts=n, extra_tokens=qt.numel())
    d_qt, d_qo, d_arr = dev(qt), dev(qo), dev(w.arrivals)
    ks = [1, 2, 4, 8]
    trees = [K.rt_clone(base) for _ in ks]
    torch.cuda.synchronize()
    streams = [torch.cuda.Stream() for _ in ks]
    outs = []
    for k, tree, st in zip(ks, trees, streams):
        with torch.cuda.stream(st):
            order = torch.full((n,), -1, dtype=torch.int32, device="cuda")
            unc = torch.full((n,), -1, dtype=torch.int32, device="cuda")
            ttft = torch.full((n,), -1, dtype=torch.int64, device="cuda")
            comp = torch.full((n,), -1, dtype=torch.int64, device="cuda")
            K.klpm_run(tree, d_qt, d_qo, d_arr, K.make_params(K.POLICY_KLPM, k, 0, 1, w.start_tick), order, unc, ttft, comp)
            outs.append((order, unc, ttft, comp))
    torch.cuda.synchronize()
    for k, tree, (order, unc, ttft, comp) in zip(ks, trees, outs):
        assert K.rt_sync_status(tree) == 0
        got = (order.cpu().numpy(), unc.cpu().numpy(), ttft.cpu().numpy(), comp.cpu().numpy(), K.rt_stats(tree))
        want = run_oracle(pt, po, qt, qo, w.arrivals, oracle.POLICY_KLPM, k, start=w.start_tick)
        assert_same_schedule(got, want)
    # the tree the clones were taken from is untouched
    m, _, _ = gpu_match(K, base, qt, qo)
    assert np.array_equal(m, oracle_tree(pt, po).match(qt.numpy(), qo.numpy()))


# ------------------------------------------------------------------ tie priorities and the hit-rate score

def run_gpu_ex(K, pt, po, qt, qo, arr, policy, k, prio, score_mode, budget=0, start=0):
    n = qo.numel() - 1
    tree = gpu_tree(K, pt, po, extra_prompts=n, extra_tokens=qt.numel(), budget=budget)
    order = torch.full((n,), -1, dtype=torch.int32, device="cuda")
    unc = torch.full((n,), -1, dtype=torch.int32, device="cuda")
    ttft = torch.full((n,), -1, dtype=torch.int64, device="cuda")
    comp = torch.full((n,), -1, dtype=torch.int64, device="cuda")
    d_prio = None if prio is None else dev(torch.as_tensor(prio, dtype=torch.int64))
    K.klpm_run_ex(tree, dev(qt), dev(qo), dev(torch.as_tensor(arr, dtype=torch.int64)), K.make_params(policy, k, 0, 1, start),
                  d_prio, score_mode, order, unc, ttft, comp)
    assert K.rt_sync_status(tree) == 0
    st = K.rt_stats(tree)
    K.rt_destroy(tree)
    return order.cpu().numpy(), unc.cpu().numpy(), ttft.cpu().numpy(), comp.cpu().numpy(), st


def run_oracle_ex(pt, po, qt, qo, arr, policy, k, prio, score_mode, budget=0, start=0, tier=oracle.TIER_UPDATE):
    ot = oracle_tree(pt, po, budget)
    out = oracle.schedule(qt.numpy(), qo.numpy(), np.asarray(arr, dtype=np.int64), policy, k, 0, 1, start,
                          oracle.CACHE_TREE, tier, ot, prio, score_mode)
    return out + (ot.stats(),)


def test_run_ex_toy_queue_with_priorities(K):
    prompts, arr = W.regular_arrival_shuffled_queue(4, 2, 5, 5, 0, [1, 2, 3, 4])
    qt, qo = csr(prompts)
    e = torch.zeros(0, dtype=torch.int32), torch.zeros(1, dtype=torch.int64)
    order, unc, ttft, comp, _ = run_gpu_ex(K, *e, qt, qo, arr, K.POLICY_LPM, 1, [3, 2, 0, 1], 0)
    assert order.tolist() == [2, 0, 3, 1] and ttft.tolist() == [15, 30, 10, 25]


@pytest.mark.parametrize("seed", range(4))
@pytest.mark.parametrize("score_mode", [0, 1])
def test_run_ex_fuzz(K, seed, score_mode):
    prompts, arr = W.random_small_queue(seed + 1200, 150, vocab=2, max_len=14, min_len=0, max_gap=4)
    prefill, _ = W.random_small_queue(seed + 1300, 10, vocab=2, max_len=10, min_len=1)
    prio = W.uniform_int(seed, 78, len(prompts), 0, 9).tolist()
    qt, qo = csr(prompts)
    pt, po = csr(prefill)
    for policy, k in ((1, 1), (2, 3)):
        for budget in (0, 48):
            for p in (prio, None):
                got = run_gpu_ex(K, pt, po, qt, qo, arr, policy, k, p, score_mode, budget=budget)
                want = run_oracle_ex(pt, po, qt, qo, arr, policy, k, p, score_mode, budget=budget, tier=oracle.TIER_REMATCH)
                assert_same_schedule(got, want)


@pytest.mark.parametrize("score_mode", [0, 1])
def test_run_ex_multi_cta_random_ties(K, score_mode):
    """Uniformly random tie priorities (the paper's assumption for LPM) on a queue large enough for the multi-CTA loop."""
    w = W.medium(scale=1 / 4)
    pt, po = w.prefill.materialize()
    qt, qo = w.queries.materialize()
    prio = W.uniform_u53(11, 79, w.queries.n).tolist()
    got = run_gpu_ex(K, pt, po, qt, qo, w.arrivals, K.POLICY_LPM, 1, prio, score_mode, start=w.start_tick)
    want = run_oracle_ex(pt, po, qt, qo, w.arrivals, oracle.POLICY_LPM, 1, prio, score_mode, start=w.start_tick)
    assert_same_schedule(got, want)
    assert not np.array_equal(got[0], run_oracle(pt, po, qt, qo, w.arrivals, oracle.POLICY_LPM, 1, start=w.start_tick)[0])


# ------------------------------------------------------------------ bounded waits and guarded scores

def test_a_wait_that_runs_out_is_reported_and_every_cta_returns(K):
    """The CTAs of the one-decision-at-a-time loop wait for one another with a limit.  With the limit set to zero the
    sequencer gives up on its first hand-over: the call returns, the status word says RT_ERR_LIMIT (detail 102), and
    after a rollback the tree answers matches as before.  Nothing traps or hangs: a wait that gives up returns."""
    prompts, arr = W.random_small_queue(77, 6000, vocab=3, max_len=24, min_len=1, max_gap=0)      # everybody waiting
    prefill, _ = W.random_small_queue(78, 50, vocab=3, max_len=20, min_len=1)
    qt, qo = csr(prompts)
    pt, po = csr(prefill)
    n = len(prompts)
    tree = gpu_tree(K, pt, po, extra_prompts=n, extra_tokens=qt.numel(), budget=200000)
    K.rt_checkpoint(tree)
    out = [torch.full((n,), -1, dtype=torch.int32, device="cuda"), torch.full((n,), -1, dtype=torch.int32, device="cuda"),
           torch.full((n,), -1, dtype=torch.int64, device="cuda")]
    K.klpm_debug_set("wait_limit_ns", 0)
    K.klpm_debug_set("run_one_by_one", 1)
    try:
        K.klpm_run(tree, dev(qt), dev(qo), dev(torch.tensor(arr)), K.make_params(K.POLICY_KLPM, 3), *out)
        assert K.rt_sync_status(tree) == K.RT_ERR_LIMIT
        assert K.rt_status_detail(tree) == 102
        assert K.klpm_run_path(tree) == K.RUN_PATH_ONE_BY_ONE
    finally:
        K.klpm_debug_set("wait_limit_ns", -1)
    K.rt_rollback(tree)
    assert K.rt_sync_status(tree) == 0
    ot = oracle_tree(pt, po, 200000)
    assert_match_equals_oracle(K, tree, ot, qt, qo)
    # and with the default limit the same call completes and equals the oracle
    try:
        K.klpm_run(tree, dev(qt), dev(qo), dev(torch.tensor(arr)), K.make_params(K.POLICY_KLPM, 3), *out)
    finally:
        K.klpm_debug_set("run_one_by_one", -1)
    assert K.rt_sync_status(tree) == 0
    want = oracle.schedule(qt.numpy(), qo.numpy(), np.asarray(arr), oracle.POLICY_KLPM, 3, 0, 1, 0, oracle.CACHE_TREE,
                           oracle.TIER_UPDATE, ot)
    assert np.array_equal(out[0].cpu().numpy(), want[0]) and np.array_equal(out[2].cpu().numpy(), want[2])
    K.rt_destroy(tree)


def test_a_grid_barrier_that_runs_out_is_reported_too(K):
    """The concurrent insertion's later rounds run in one cooperative kernel whose CTAs meet at barriers with the same
    limit.  Prompts that share prefixes need several rounds; with the limit at zero the first barrier gives up, the
    status word says RT_ERR_LIMIT (detail 112), every CTA returns, and the same insertion goes through afterwards."""
    prompts, _ = W.random_small_queue(79, 3000, vocab=2, max_len=30, min_len=1)
    pt, po = csr(prompts)
    tree = K.rt_create(**caps(pt.numel(), n_prompts=len(prompts)))
    K.rt_checkpoint(tree)
    K.klpm_debug_set("wait_limit_ns", 0)
    try:
        K.rt_insert(tree, dev(pt), dev(po))
        assert K.rt_sync_status(tree) == K.RT_ERR_LIMIT and K.rt_status_detail(tree) == 112
    finally:
        K.klpm_debug_set("wait_limit_ns", -1)
    K.rt_rollback(tree)
    K.rt_insert(tree, dev(pt), dev(po))
    assert K.rt_sync_status(tree) == 0
    ot = oracle_tree(pt, po)
    st, ost = K.rt_stats(tree), ot.stats()
    assert (st["n_nodes"], st["tokens"], st["clock"]) == (ost["n_nodes"], ost["tokens"], ost["clock"])
    assert_match_equals_oracle(K, tree, ot, pt, po)
    K.rt_destroy(tree)


def test_hit_rate_score_refuses_prompts_it_cannot_order_exactly(K):
    """The hit-rate key orders prompts exactly as the rates m/|x| do up to 46,340 tokens per prompt; one longer
    prompt makes the status word say so (both loops)."""
    prompts = [[1] + [2] * 46340, [1, 3, 4]]
    qt, qo = csr(prompts)
    for budget in (0, 1 << 20):
        tree = K.rt_create(budget_tokens=budget, **caps(qt.numel(), n_prompts=2))
        out = [torch.zeros(2, dtype=torch.int32, device="cuda"), torch.zeros(2, dtype=torch.int32, device="cuda"),
               torch.zeros(2, dtype=torch.int64, device="cuda")]
        K.klpm_run_ex(tree, dev(qt), dev(qo), dev(torch.zeros(2, dtype=torch.int64)), K.make_params(K.POLICY_LPM), None, 1, *out)
        assert K.rt_sync_status(tree) == K.RT_ERR_INVALID and K.rt_status_detail(tree) == 109
        K.rt_destroy(tree)
        tree = K.rt_create(budget_tokens=budget, **caps(qt.numel(), n_prompts=2))
        K.klpm_run_ex(tree, dev(qt), dev(qo), dev(torch.zeros(2, dtype=torch.int64)), K.make_params(K.POLICY_LPM), None, 0, *out)
        assert K.rt_sync_status(tree) == 0
        K.rt_destroy(tree)
