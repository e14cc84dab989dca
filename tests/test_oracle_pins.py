"""Pins for the CPU oracle: values the paper prints, closed forms from its proofs,
brute force from the definitions, and limits the paper states.  No GPU involved."""
import itertools
import math
import os

import numpy as np
import pytest

import oracle
from oracle import definition as D
from paper_2502_04677_b200 import workloads as W

GOLDEN = os.path.join(os.path.dirname(__file__), "golden")


def csr(prompts):
    t, o = W.to_csr(prompts)
    return t.numpy(), o.numpy()


def run(prompts, arrivals, policy, k=1, mode=oracle.CACHE_TREE, tier=oracle.TIER_UPDATE, start=0,
        c_num=0, c_den=1, budget=0, prefill=(), indexed=True):
    t, o = csr(prompts)
    tree = None
    if mode == oracle.CACHE_TREE:
        tree = oracle.OracleTree(budget, indexed)
        if len(prefill):
            tree.insert(*csr(prefill))
    order, unc, ttft, comp = oracle.schedule(t, o, arrivals, policy, k, c_num, c_den, start, mode, tier, tree)
    return order.tolist(), unc.tolist(), ttft.tolist(), comp.tolist()


# ---------------------------------------------------------------- overlap / match

def test_overlap_definition():
    assert oracle.overlap([1, 2, 3], [1, 2, 4]) == 2
    assert oracle.overlap([], [1]) == 0
    assert oracle.overlap([1, 2], [1, 2, 3]) == 2
    assert oracle.overlap([5], [6]) == 0
    assert D.overlap([1, 2, 3], [1, 2, 4]) == 2


@pytest.mark.parametrize("seed", range(6))
def test_tree_match_equals_bruteforce_lcp(seed):
    """Tree walk == max over every cached prompt of overlap (brute force, two independent codes)."""
    cached, _ = W.random_small_queue(seed, 60, vocab=3, max_len=14)
    queries, _ = W.random_small_queue(seed + 100, 80, vocab=3, max_len=18)
    ct, co = csr(cached)
    qt, qo = csr(queries)
    tree = oracle.OracleTree()
    tree.insert(ct, co)
    got = tree.match(qt, qo)
    brute = oracle.match_bruteforce(qt, qo, ct, co)
    py = [max([D.overlap(q, c) for c in cached] + [0]) for q in queries]
    assert got.tolist() == brute.tolist() == py
    assert tree.match(qt, qo, threads=3).tolist() == py
    # invariants: 0 <= m <= |x|
    assert all(0 <= m <= len(q) for m, q in zip(py, queries))


def test_match_invariants():
    cached, _ = W.random_small_queue(7, 40, vocab=2, max_len=12, min_len=1)
    ct, co = csr(cached)
    tree = oracle.OracleTree()
    new = tree.insert(ct, co)
    # a processed prompt is fully cached afterwards
    assert tree.match(ct, co).tolist() == [len(c) for c in cached]
    # tokens held = number of distinct non-empty prefixes = sum of new tokens
    distinct = {tuple(c[:i]) for c in cached for i in range(1, len(c) + 1)}
    assert tree.stats()["tokens"] == len(distinct) == int(new.sum())
    # match(q, S + p) = max(match(q, S), overlap(q, p))
    queries, _ = W.random_small_queue(8, 30, vocab=2, max_len=12)
    qt, qo = csr(queries)
    before = tree.match(qt, qo)
    p = [0, 1, 1, 0, 1, 0, 0, 1, 1, 1, 0, 1, 0]
    tree.insert(*csr([p]))
    after = tree.match(qt, qo)
    assert after.tolist() == [max(int(b), D.overlap(q, p)) for b, q in zip(before, queries)]


@pytest.mark.parametrize("seed", range(6))
@pytest.mark.parametrize("budget", [0, 36])
def test_where_a_match_ends_against_the_string_set_model(seed, budget):
    """The edge that holds the last matched token: how far into it the match goes and how deep it starts.
    Pointer tree vs the set-of-strings model (node = shortest node-end string extending the matched part)."""
    cached, _ = W.random_small_queue(seed + 700, 50, vocab=2, max_len=13, min_len=1)
    queries, _ = W.random_small_queue(seed + 800, 70, vocab=2, max_len=16)
    model = D.StringSetCache(budget)
    tree = oracle.OracleTree(budget)
    for p in cached:
        model.process(p)
        tree.insert(*csr([p]))
    m, off, depth = tree.match_pos(*csr(queries))
    want = [model.match_pos(q) for q in queries]
    assert list(zip(m.tolist(), off.tolist(), depth.tolist())) == want
    assert m.tolist() == tree.match(*csr(queries)).tolist()
    assert any(0 < o for _, o, _ in want) and any(d > 0 for _, _, d in want)
    if budget:
        assert model.evictions > 0


def test_where_a_match_ends_by_hand():
    """Tree of "abcd" and "abxy": nodes "ab" (depth 0), "cd" and "xy" (depth 2)."""
    tree = oracle.OracleTree()
    tree.insert(*csr([[1, 2, 3, 4], [1, 2, 7, 8]]))
    qs = [[1], [1, 2], [1, 2, 3], [1, 2, 7, 8, 9], [5], [], [1, 2, 9]]
    m, off, depth = tree.match_pos(*csr(qs))
    assert m.tolist() == [1, 2, 3, 4, 0, 0, 2]
    assert off.tolist() == [1, 2, 1, 2, 0, 0, 2]
    assert depth.tolist() == [0, 0, 2, 2, 0, 0, 0]


# ---------------------------------------------------------------- the printed toy example

def _read_toy():
    rows = []
    for line in open(os.path.join(GOLDEN, "toy_example.txt")):
        if line.startswith("#") or not line.strip():
            continue
        s, pol, order, ttft = line.split()
        rows.append((int(s.split("=")[1]), pol, [int(v) - 1 for v in order.split("=")[1].split(",")],
                     [int(v) for v in ttft.split("=")[1].split(",")]))
    return rows


@pytest.mark.parametrize("tier", [oracle.TIER_REMATCH, oracle.TIER_UPDATE])
def test_toy_example_printed_values(tier):
    for s, pol, order, ttft in _read_toy():
        prompts, arr = W.regular_arrival_shuffled_queue(4, 2, 5, 5, s, [1, 2, 3, 4])
        policy = {"FCFS": oracle.POLICY_FCFS, "LPM": oracle.POLICY_LPM}[pol]
        got = run(prompts, arr, policy, mode=oracle.CACHE_LAST_ONLY, tier=tier)
        assert got[0] == order and got[2] == ttft, (s, pol, got)
        assert D.schedule(prompts, arr, policy, cache_mode=D.LAST_ONLY)[0] == order
        assert D.schedule(prompts, arr, policy, cache_mode=D.LAST_ONLY)[2] == ttft
    # k-LPM with k = 2 on the burst case: oldest, best match, oldest, best match
    prompts, arr = W.regular_arrival_shuffled_queue(4, 2, 5, 5, 0, [1, 2, 3, 4])
    for mode in (oracle.CACHE_LAST_ONLY, oracle.CACHE_TREE):
        o, u, t, c = run(prompts, arr, oracle.POLICY_KLPM, k=2, mode=mode, tier=tier)
        assert o == [0, 2, 1, 3] and max(t) == 30 and u == [10, 10, 5, 5]
    # with the whole tree cached FCFS reuses user1 for x3 although x2 came in between
    assert run(prompts, arr, oracle.POLICY_FCFS, mode=oracle.CACHE_TREE)[2] == [10, 20, 25, 30]


# ---------------------------------------------------------------- one decision as a function of a snapshot

def test_select_by_hand_and_against_the_definition():
    """Toy queue after x1 was processed: x3 shares x1's user (match 5), the others match 0.  The longest-match turn
    takes x3, the oldest-first turn x2; among equal matches the earliest arrival wins, among equal arrivals the
    lower index; nobody waiting gives -1."""
    m, t, w = [10, 0, 5, 0], [0, 0, 0, 0], [0, 1, 1, 1]
    assert oracle.select(m, t, w, 1, oracle.POLICY_KLPM, 2) == 2        # turn 1 of a 2-cycle: longest match
    assert oracle.select(m, t, w, 2, oracle.POLICY_KLPM, 2) == 1        # turn 2: the oldest waiting
    assert oracle.select(m, t, w, 7, oracle.POLICY_FCFS) == 1
    assert oracle.select(m, t, w, 0, oracle.POLICY_LPM) == 2
    assert oracle.select([3, 3, 3], [5, 2, 2], [1, 1, 1], 1, oracle.POLICY_LPM) == 1
    assert oracle.select([3, 3], [5, 2], [0, 0], 1, oracle.POLICY_LPM) == -1
    rng = np.random.RandomState(0)
    for _ in range(200):
        n = int(rng.randint(1, 40))
        m, t, w = rng.randint(0, 4, n), rng.randint(0, 5, n), rng.randint(0, 2, n)
        for policy, k, c in ((0, 1, 3), (1, 1, 3), (2, 3, 0), (2, 3, 1), (2, 3, 5), (2, 1, 4)):
            assert oracle.select(m, t, w, c, policy, k) == D.select(m.tolist(), t.tolist(), w.tolist(), c, policy, k)
    # the loop's own picks are this rule applied to the match lengths of the moment
    prompts, arr = W.regular_arrival_shuffled_queue(4, 2, 5, 5, 0, [1, 2, 3, 4])
    order = run(prompts, arr, oracle.POLICY_KLPM, k=2, mode=oracle.CACHE_LAST_ONLY)[0]
    assert order[1] == oracle.select([0, 0, 5, 0], arr, [0, 1, 1, 1], 1, oracle.POLICY_KLPM, 2)


# ---------------------------------------------------------------- limits of k-LPM

@pytest.mark.parametrize("seed", range(5))
@pytest.mark.parametrize("mode", [oracle.CACHE_LAST_ONLY, oracle.CACHE_TREE])
def test_k1_is_fcfs_and_k_infinite_is_lpm(seed, mode):
    prompts, arr = W.random_small_queue(seed, 24, vocab=2, max_len=10, min_len=1)
    n = len(prompts)
    fcfs = run(prompts, arr, oracle.POLICY_FCFS, mode=mode)
    k1 = run(prompts, arr, oracle.POLICY_KLPM, k=1, mode=mode)
    assert fcfs == k1
    # FCFS order is the arrival order (ties: lower index)
    assert fcfs[0] == sorted(range(n), key=lambda i: (arr[i], i))
    # k larger than the stream, empty cache: Algorithm 1's first pick is the oldest query, which is
    # also LPM's pick when nothing is cached; every later pick is a longest-match pick
    lpm = run(prompts, arr, oracle.POLICY_LPM, mode=mode)
    kinf = run(prompts, arr, oracle.POLICY_KLPM, k=n + 1, mode=mode)
    assert lpm == kinf


@pytest.mark.parametrize("k", [2, 3, 5])
def test_every_kth_pick_is_the_oldest_waiting(k):
    prompts, arr = W.random_small_queue(11, 40, vocab=2, max_len=12, min_len=1, max_gap=6)
    order, unc, ttft, comp = run(prompts, arr, oracle.POLICY_KLPM, k=k)
    done = set()
    now = 0
    for c, j in enumerate(order):
        waiting = [i for i in range(len(prompts)) if i not in done and arr[i] <= now]
        if not waiting:
            now = min(arr[i] for i in range(len(prompts)) if i not in done)
            waiting = [i for i in range(len(prompts)) if i not in done and arr[i] <= now]
        assert j in waiting
        if c % k == 0:
            assert j == min(waiting, key=lambda i: (arr[i], i))
        done.add(j)
        now = comp[j]


# ---------------------------------------------------------------- closed forms (proof of Theorem 2)

@pytest.mark.parametrize("n,rep,u,d,s", [(6, 2, 4, 3, 1), (6, 3, 5, 2, 2), (8, 2, 3, 3, 1), (12, 4, 6, 1, 2)])
@pytest.mark.parametrize("mode", [oracle.CACHE_LAST_ONLY, oracle.CACHE_TREE])
def test_lpm_closed_form_completion(n, rep, u, d, s, mode):
    """All arrived by T, empty cache: the j-th processed query completes at T + ceil(j/rep) u + j d."""
    rng = np.random.RandomState(n * 100 + rep)
    for _ in range(5):
        sigma = (rng.permutation(n) + 1).tolist()
        prompts, arr = W.regular_arrival_shuffled_queue(n, rep, u, d, s, sigma)
        T = s * n
        order, unc, ttft, comp = run(prompts, arr, oracle.POLICY_LPM, mode=mode, start=T)
        for pos, j in enumerate(order, start=1):
            assert comp[j] == T + math.ceil(pos / rep) * u + d * pos
            assert ttft[j] + arr[j] == comp[j]


@pytest.mark.parametrize("n,rep,u,d,s", [(6, 2, 4, 3, 1), (8, 4, 6, 1, 2), (12, 3, 5, 2, 1)])
def test_fcfs_closed_form_last_query(n, rep, u, d, s):
    """Last-prompt cache: TTFT_n = T + n(u+d) - s n - u sum_i I_i, I_i = consecutive arrivals share a user."""
    rng = np.random.RandomState(n + rep)
    for _ in range(8):
        sigma = (rng.permutation(n) + 1).tolist()
        prompts, arr = W.regular_arrival_shuffled_queue(n, rep, u, d, s, sigma)
        T = s * n
        order, unc, ttft, comp = run(prompts, arr, oracle.POLICY_FCFS, mode=oracle.CACHE_LAST_ONLY, start=T)
        by_arrival = sorted(range(n), key=lambda i: arr[i])
        I = sum(1 for a, b in zip(by_arrival, by_arrival[1:]) if prompts[a][0] == prompts[b][0])
        assert ttft[by_arrival[-1]] == T + n * (u + d) - s * n - u * I


@pytest.mark.parametrize("n,rep,u,d,s", [(6, 2, 4, 3, 1), (6, 3, 5, 2, 2)])
def test_klpm_bound_every_permutation(n, rep, u, d, s):
    """k = rep, T >= s n: max TTFT <= T + n(u/k + d - s/k) for every arrival order (Theorem 2, k-LPM part);
    all queries are done by T + n(u/k + d) and the i-th arrival by T + i(u + k d)."""
    T = s * n
    for perm in itertools.permutations(range(1, n + 1)):
        prompts, arr = W.regular_arrival_shuffled_queue(n, rep, u, d, s, list(perm))
        order, unc, ttft, comp = run(prompts, arr, oracle.POLICY_KLPM, k=rep, mode=oracle.CACHE_LAST_ONLY, start=T)
        assert max(ttft) * rep <= T * rep + n * (u + rep * d - s)
        assert max(comp) * rep <= T * rep + n * (u + rep * d)
        for i in range(n):
            assert comp[i] <= T + (arr[i] // s) * (u + rep * d)


def test_klpm_bound_random_large():
    n, rep, u, d, s = 240, 4, 9, 3, 2
    rng = np.random.RandomState(5)
    T = s * n
    for mode in (oracle.CACHE_LAST_ONLY, oracle.CACHE_TREE):
        for _ in range(3):
            sigma = (rng.permutation(n) + 1).tolist()
            prompts, arr = W.regular_arrival_shuffled_queue(n, rep, u, d, s, sigma)
            _, _, ttft, _ = run(prompts, arr, oracle.POLICY_KLPM, k=rep, mode=mode, start=T)
            assert max(ttft) * rep <= T * rep + n * (u + rep * d - s)


# ---------------------------------------------------------------- offline optimality of LPM

@pytest.mark.parametrize("seed", range(12))
def test_offline_lpm_maximises_reuse_exhaustive(seed):
    """Uniform arrivals, last-prompt cache, n <= 7: no processing order reuses more tokens than LPM."""
    n = 5 + seed % 3
    prompts, _ = W.random_small_queue(seed + 40, n, vocab=2, max_len=7, min_len=1)
    arr = [0] * n
    _, unc, _, _ = run(prompts, arr, oracle.POLICY_LPM, mode=oracle.CACHE_LAST_ONLY)
    total = sum(len(p) for p in prompts)
    lpm_reuse = total - sum(unc)
    best = 0
    for perm in itertools.permutations(range(n)):
        reuse = sum(D.overlap(prompts[a], prompts[b]) for a, b in zip(perm, perm[1:]))
        best = max(best, reuse)
    assert lpm_reuse == best


@pytest.mark.parametrize("seed", range(4))
def test_tree_cache_total_uncached_is_order_independent(seed):
    """Unbounded tree cache: sum of uncached tokens = number of distinct non-empty prefixes, any policy."""
    prompts, arr = W.random_small_queue(seed + 60, 30, vocab=3, max_len=10)
    distinct = {tuple(p[:i]) for p in prompts for i in range(1, len(p) + 1)}
    for policy, k in ((oracle.POLICY_FCFS, 1), (oracle.POLICY_LPM, 1), (oracle.POLICY_KLPM, 3)):
        _, unc, _, _ = run(prompts, arr, policy, k=k)
        assert sum(unc) == len(distinct)


# ---------------------------------------------------------------- the NP-hardness gadget, worked by hand

def test_three_partition_gadget_feasible_order():
    rows = [l.split() for l in open(os.path.join(GOLDEN, "three_partition_gadget.txt"))
            if l.strip() and not l.startswith("#")]
    a = [5, 5, 6, 5, 5, 6]
    prompts, arr, T, labels = W.three_partition_gadget(a, 2, 16)
    assert T == 96
    xs = [i for i, l in enumerate(labels) if l == "x"]
    idx = {l: i for i, l in enumerate(labels) if l != "x"}
    order = [idx["w1"], xs[0], xs[1], xs[2], idx["y1"], idx["z1"], xs[3], xs[4], xs[5], idx["y2"], idx["z2"], idx["w2"]]
    t, o = csr(prompts)
    unc, ttft, comp = oracle.replay(order, t, o, arr, cache_mode=oracle.CACHE_LAST_ONLY)
    for j, row in zip(order, rows):
        label, arrival, length, completion, tt = row[0], int(row[1]), int(row[2]), int(row[3]), int(row[4])
        assert labels[j] == label and arr[j] == arrival and len(prompts[j]) == length
        assert comp[j] == completion and ttft[j] == tt
    assert max(ttft) == T
    assert unc[idx["z1"]] == 0 and unc[idx["z2"]] == 0          # identical prompt right after its twin is free
    assert D.replay(order, prompts, arr, cache_mode=D.LAST_ONLY)[1] == ttft.tolist()
    # a non-partition order (x's not in groups summing to H) breaks the constraint
    bad = [idx["w1"], xs[0], xs[1], xs[3], idx["y1"], idx["z1"], xs[2], xs[5], xs[4], idx["y2"], idx["z2"], idx["w2"]]
    assert max(oracle.replay(bad, t, o, arr, cache_mode=oracle.CACHE_LAST_ONLY)[1]) > T


# ---------------------------------------------------------------- Definition 2 along a fixed order, tree cache

def test_replay_with_the_tree_cache_by_hand():
    """Budget 6, order 0,1,2,3.  111 and 222 fill the cache (R = 3, 6).  115 matches "11": the edge 111 is cut,
    the stale lower "1" is the oldest leaf and goes (1 token), leaf "5" is charged 1 token (R = 7).  333 arrives at
    20: 222 is evicted, processing starts at 20 (R = 23, TTFT 3)."""
    prompts, arr = [[1, 1, 1], [2, 2, 2], [1, 1, 5], [3, 3, 3]], [0, 0, 0, 20]
    t, o = csr(prompts)
    tree = oracle.OracleTree(6)
    unc, ttft, comp = oracle.replay([0, 1, 2, 3], t, o, arr, cache_mode=oracle.CACHE_TREE, tree=tree)
    assert unc.tolist() == [3, 3, 1, 3] and comp.tolist() == [3, 6, 7, 23] and ttft.tolist() == [3, 6, 7, 3]
    assert tree.stats() == dict(n_nodes=3, tokens=6, clock=4, evictions=2)
    assert tree.match(*csr([[1, 1, 1], [2, 2, 2], [1, 1, 5], [3, 3, 3]])).tolist() == [2, 0, 3, 3]
    # c_attn = 1/2, times in half ticks: cost = (2 + |x|)(|x| - m)
    unc, ttft, comp = oracle.replay([0, 1, 2, 3], t, o, arr, 1, 2, 0, oracle.CACHE_TREE, oracle.OracleTree(6))
    assert comp.tolist() == [15, 30, 35, 50] and ttft.tolist() == [15, 30, 35, 30]
    # queries that are not in the order keep their zeros; a later start delays everything
    unc, ttft, comp = oracle.replay([2, 0], t, o, arr, 0, 1, 100, oracle.CACHE_TREE, oracle.OracleTree(6))
    assert unc.tolist() == [1, 0, 3, 0] and comp.tolist() == [104, 0, 103, 0]


@pytest.mark.parametrize("seed", range(8))
@pytest.mark.parametrize("budget", [0, 30])
def test_replay_with_the_tree_cache_against_the_definition(seed, budget):
    """Random orders (a permutation, and a partial order with a repeat-free subset) over a pre-filled cache."""
    prompts, arr = W.random_small_queue(seed + 1000, 24, vocab=2, max_len=12, min_len=1, max_gap=5)
    prefill, _ = W.random_small_queue(seed + 1100, 5, vocab=2, max_len=9, min_len=1)
    rng = np.random.RandomState(seed)
    perm = rng.permutation(len(prompts)).tolist()
    for order in (perm, perm[:11]):
        for c_num, c_den in ((0, 1), (1, 3)):
            tree = oracle.OracleTree(budget)
            tree.insert(*csr(prefill))
            got = oracle.replay(order, *csr(prompts), arr, c_num, c_den, 2, oracle.CACHE_TREE, tree)
            ref = D.replay(order, prompts, arr, c_num, c_den, 2, D.TREE, prefill=prefill, budget=budget)
            assert [g.tolist() for g in got] == [list(r) for r in ref]


# ---------------------------------------------------------------- cost model details

def test_cost_model_first_query_and_c_attn():
    """R(j_1) = |x| + c |x|^2 (Definition 2); with c = 1/2 and times in half ticks: (2 + |x|)|x|."""
    prompts, arr = [[1, 2, 3, 4], [1, 2, 9, 9, 9, 9]], [0, 0]
    o, unc, ttft, comp = run(prompts, arr, oracle.POLICY_FCFS, c_num=1, c_den=2, mode=oracle.CACHE_LAST_ONLY)
    assert comp[0] == (2 + 4) * 4                      # = 2 * (4 + 0.5 * 16)
    assert comp[1] == comp[0] + (2 + 6) * (6 - 2)      # (1 + c|x|)(|x| - overlap), in half ticks
    # arrival gating: a query cannot start before it arrives
    o, unc, ttft, comp = run([[1], [2]], [0, 50], oracle.POLICY_FCFS)
    assert comp == [1, 51] and ttft == [1, 1]


# ---------------------------------------------------------------- tiers and the definition-level model agree

@pytest.mark.parametrize("seed", range(8))
@pytest.mark.parametrize("budget", [0, 40])
def test_tiers_and_definition_agree(seed, budget):
    prompts, arr = W.random_small_queue(seed + 200, 28, vocab=2, max_len=12, min_len=1, max_gap=4)
    prefill, _ = W.random_small_queue(seed + 300, 6, vocab=2, max_len=10, min_len=1)
    for policy, k in ((oracle.POLICY_FCFS, 1), (oracle.POLICY_LPM, 1), (oracle.POLICY_KLPM, 2), (oracle.POLICY_KLPM, 4)):
        ref = D.schedule(prompts, arr, policy, k, prefill=prefill, budget=budget)
        for tier in (oracle.TIER_REMATCH, oracle.TIER_UPDATE):
            for indexed in (True, False):
                got = run(prompts, arr, policy, k, tier=tier, budget=budget, prefill=prefill, indexed=indexed)
                assert got[0] == ref[0] and got[1] == ref[1] and got[2] == ref[2] and got[3] == ref[3]
        ref_last = D.schedule(prompts, arr, policy, k, cache_mode=D.LAST_ONLY)
        for tier in (oracle.TIER_REMATCH, oracle.TIER_UPDATE):
            got = run(prompts, arr, policy, k, mode=oracle.CACHE_LAST_ONLY, tier=tier)
            assert list(got) == [list(v) for v in ref_last]


@pytest.mark.parametrize("seed", range(6))
def test_lru_against_string_set_model(seed):
    """Eviction order and sizes: pointer tree (ordered index and linear scan) vs the set-of-strings model."""
    prompts, _ = W.random_small_queue(seed + 400, 60, vocab=2, max_len=14, min_len=1)
    budget = 30
    model = D.StringSetCache(budget)
    trees = [oracle.OracleTree(budget, True), oracle.OracleTree(budget, False)]
    for p in prompts:
        u = model.process(p)
        for t in trees:
            new = t.insert(*csr([p]))
            st = t.stats()
            assert int(new[0]) == u
            assert st["tokens"] == model.tokens() <= budget
            assert st["evictions"] == model.evictions
            assert st["n_nodes"] == len(model.nodes)
    assert model.evictions > 0
    qs, _ = W.random_small_queue(seed + 500, 40, vocab=2, max_len=14)
    for t in trees:
        assert t.match(*csr(qs)).tolist() == [model.match(q) for q in qs]


def test_lru_evicts_least_recently_used_leaf_by_hand():
    """Budget 6.  aaa, bbb fill it; ccc evicts aaa (oldest); touching bbb then adding ddd evicts ccc."""
    t = oracle.OracleTree(6)
    seq = [[1, 1, 1], [2, 2, 2], [3, 3, 3], [2, 2, 2], [4, 4, 4]]
    new = [int(t.insert(*csr([p]))[0]) for p in seq]
    assert new == [3, 3, 3, 0, 3]
    assert t.match(*csr([[1, 1, 1], [2, 2, 2], [3, 3, 3], [4, 4, 4]])).tolist() == [0, 3, 0, 3]
    with pytest.raises(RuntimeError):
        oracle.OracleTree(2).insert(*csr([[1, 2, 3]]))


# ---------------------------------------------------------------- batch size B (Section 2.1)

def test_batch_times_by_hand_and_limits():
    """Toy example under LPM: order x1,x3,x2,x4 completes at 10,15,25,30; with B = 2 the bins finish at 15 and 30."""
    order = [0, 2, 1, 3]
    comp = np.array([10, 25, 15, 30], dtype=np.int64)          # indexed by query
    arr = [0, 0, 0, 0]
    ttft, cb = oracle.batch_times(order, arr, comp, 2)
    assert cb.tolist() == [15, 30, 15, 30] and ttft.tolist() == [15, 30, 15, 30]
    assert oracle.batch_times(order, arr, comp, 1)[1].tolist() == comp.tolist()       # B = 1 changes nothing
    assert oracle.batch_times(order, arr, comp, 9)[1].tolist() == [30] * 4            # one bin: everyone waits for the last
    ttft, cb = oracle.batch_times(order, [0, 5, 1, 2], comp, 3)                       # ragged last bin, arrivals subtracted
    assert cb.tolist() == [25, 25, 25, 30] and ttft.tolist() == [25, 20, 24, 28]


# ---------------------------------------------------------------- tie priorities and the hit-rate score

def run_ex(prompts, arrivals, policy, k=1, prio=None, score_mode=0, tier=oracle.TIER_UPDATE, start=0, budget=0):
    t, o = csr(prompts)
    tree = oracle.OracleTree(budget)
    out = oracle.schedule(t, o, arrivals, policy, k, 0, 1, start, oracle.CACHE_TREE, tier, tree, prio, score_mode)
    return [v.tolist() for v in out]


def test_tie_priorities_by_hand_on_the_toy_queue():
    """Toy queue, burst: every first pick is a tie.  With priorities that favour x3, then x4: LPM processes
    x3, x1 (same user as x3), x4, x2 and the completions are 10, 15, 25, 30 in that order."""
    prompts, arr = W.regular_arrival_shuffled_queue(4, 2, 5, 5, 0, [1, 2, 3, 4])
    order, unc, ttft, comp = run_ex(prompts, arr, oracle.POLICY_LPM, prio=[3, 2, 0, 1])
    assert order == [2, 0, 3, 1] and ttft == [15, 30, 10, 25] and unc == [5, 5, 10, 10]
    # priorities that repeat the arrival order change nothing
    base = run_ex(prompts, arr, oracle.POLICY_LPM)
    assert run_ex(prompts, arr, oracle.POLICY_LPM, prio=[0, 1, 2, 3]) == base
    # k-LPM: the oldest-first picks ignore the priorities
    order, _, _, _ = run_ex(prompts, arr, oracle.POLICY_KLPM, k=2, prio=[3, 2, 0, 1])
    assert order == [0, 2, 1, 3]


@pytest.mark.parametrize("n,rep,u,d,s", [(12, 4, 6, 1, 2), (8, 2, 3, 3, 1)])
def test_lpm_closed_form_holds_for_random_ties(n, rep, u, d, s):
    """The j-th completion under LPM is T + ceil(j/rep) u + j d whatever breaks the ties (proof of Theorem 2)."""
    rng = np.random.RandomState(n)
    for _ in range(6):
        sigma = (rng.permutation(n) + 1).tolist()
        prompts, arr = W.regular_arrival_shuffled_queue(n, rep, u, d, s, sigma)
        prio = rng.permutation(n).tolist()
        T = s * n
        order, unc, ttft, comp = run_ex(prompts, arr, oracle.POLICY_LPM, prio=prio, start=T)
        for pos, j in enumerate(order, start=1):
            assert comp[j] == T + math.ceil(pos / rep) * u + d * pos
        # first pick of every group of `rep` is the waiting query with the smallest priority among the ties
        assert order[0] == min(range(n), key=lambda i: prio[i])


def test_hit_rate_score_by_hand_and_on_constant_lengths():
    """Cache holds "ab".  By match length "abX" and "abYZWQ" tie at 2 and beat "a"; by hit rate "a" is fully
    cached (1), then "abX" (2/3), then "abYZWQ" (1/3)."""
    cached = [[1, 2]]
    qs = [[1, 2, 7, 8, 9, 10], [1, 2, 5], [1]]
    t, o = csr(qs)
    for mode, want in ((0, [0, 1, 2]), (1, [2, 1, 0])):
        tree = oracle.OracleTree()
        tree.insert(*csr(cached))
        order = oracle.schedule(t, o, [0, 0, 0], oracle.POLICY_LPM, 1, 0, 1, 0, oracle.CACHE_TREE, oracle.TIER_REMATCH, tree,
                                None, mode)[0].tolist()
        assert order == want
    # all prompts of a regular arrival queue have the same length: both scores order them alike
    prompts, arr = W.regular_arrival_shuffled_queue(12, 3, 5, 2, 1, [5, 1, 9, 3, 12, 7, 2, 11, 4, 8, 6, 10])
    assert run_ex(prompts, arr, oracle.POLICY_KLPM, k=3, score_mode=1) == run_ex(prompts, arr, oracle.POLICY_KLPM, k=3)


def test_hit_rate_is_compared_exactly():
    """1/100000 > 1/100001 although both round to the same multiple of 2^-31: the longer prompt arrived first and
    would win a tie, the shorter one has the higher hit rate and is processed first."""
    cached = [[1]]
    a = [1] + [2] * 100000            # arrives first, hit rate 1/100001
    b = [1] + [3] * 99999             # arrives second, hit rate 1/100000
    assert (1 << 31) // len(a) == (1 << 31) // len(b)
    t, o = csr([a, b])
    for tier in (oracle.TIER_REMATCH, oracle.TIER_UPDATE):
        tree = oracle.OracleTree()
        tree.insert(*csr(cached))
        order = oracle.schedule(t, o, [0, 1], oracle.POLICY_LPM, 1, 0, 1, 5, oracle.CACHE_TREE, tier, tree, None, 1)[0]
        assert order.tolist() == [1, 0]
    assert D.schedule([a, b], [0, 1], D.LPM, start_tick=5, prefill=cached, score_mode=1)[0] == [1, 0]
    # equal rates (2/4 and 1/2, cache "12") are a tie that the earlier arrival wins; by match length 2 beats 1
    t, o = csr([[1, 2, 5, 6], [1, 7]])
    for mode, want in ((1, [1, 0]), (0, [0, 1])):
        tree = oracle.OracleTree()
        tree.insert(*csr([[1, 2]]))
        order = oracle.schedule(t, o, [1, 0], oracle.POLICY_LPM, 1, 0, 1, 5, oracle.CACHE_TREE, oracle.TIER_REMATCH, tree, None, mode)[0]
        assert order.tolist() == want


@pytest.mark.parametrize("seed", range(6))
def test_variants_agree_with_the_definition_level_model(seed):
    prompts, arr = W.random_small_queue(seed + 900, 26, vocab=2, max_len=11, min_len=0, max_gap=3)
    prio = W.uniform_int(seed, 77, len(prompts), 0, 5).tolist()          # few distinct values: ties among priorities too
    for policy, k in ((oracle.POLICY_LPM, 1), (oracle.POLICY_KLPM, 3)):
        for mode in (0, 1):
            for budget in (0, 40):
                ref = D.schedule(prompts, arr, policy, k, budget=budget, tie_priority=prio, score_mode=mode)
                for tier in (oracle.TIER_REMATCH, oracle.TIER_UPDATE):
                    got = run_ex(prompts, arr, policy, k, prio, mode, tier, budget=budget)
                    assert got == [list(v) for v in ref]
