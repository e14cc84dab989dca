"""klpm_run_last_only_batch: many independent queues under the last-prompt cache (Definition 2 as printed), one warp
each, against the CPU oracle queue by queue and against the closed forms and the bound of Theorem 2."""
import math

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


def run_batch(K, queues, arrivals, policy, k, prio=None, c_num=0, c_den=1, start=0):
    """queues: list of lists of prompts.  Returns per-queue (order, uncached, ttft, completion) and the skip count."""
    flat = [p for q in queues for p in q]
    tok, off = W.to_csr(flat)
    qoff = np.zeros(len(queues) + 1, dtype=np.int32)
    qoff[1:] = np.cumsum([len(q) for q in queues])
    arr = torch.tensor([t for a in arrivals for t in a], dtype=torch.int64)
    n = len(flat)
    d_tok = tok.cuda() if tok.numel() else torch.zeros(1, dtype=torch.int32, device="cuda")
    order = torch.full((n,), -7, dtype=torch.int32, device="cuda")
    unc = torch.full((n,), -7, dtype=torch.int32, device="cuda")
    ttft = torch.full((n,), -7, dtype=torch.int64, device="cuda")
    comp = torch.full((n,), -7, dtype=torch.int64, device="cuda")
    skipped = torch.full((1,), -7, dtype=torch.int32, device="cuda")
    d_prio = None if prio is None else torch.tensor([x for p in prio for x in p], dtype=torch.int64).cuda()
    K.klpm_run_last_only_batch(d_tok, off.cuda(), arr.cuda(), d_prio, torch.from_numpy(qoff).cuda(),
                               K.make_params(policy, k, c_num, c_den, start), order, unc, ttft, comp, skipped)
    torch.cuda.synchronize()
    o, u, t, c = order.cpu().numpy(), unc.cpu().numpy(), ttft.cpu().numpy(), comp.cpu().numpy()
    out = [(o[a:b], u[a:b], t[a:b], c[a:b]) for a, b in zip(qoff[:-1], qoff[1:])]
    return out, int(skipped.item())


def oracle_queue(prompts, arr, policy, k, prio=None, c_num=0, c_den=1, start=0):
    t, o = W.to_csr(prompts)
    return oracle.schedule(t.numpy(), o.numpy(), np.asarray(arr, dtype=np.int64), policy, k, c_num, c_den, start,
                           oracle.CACHE_LAST_ONLY, oracle.TIER_REMATCH, None, prio, 0)


def test_toy_example_on_the_device(K):
    """Section 4.2: burst (s = 0) FCFS 10, 20, 30, 40; LPM order x1, x3, x2, x4 with 10, 15, 25, 30; s = 10: all 10."""
    burst = W.regular_arrival_shuffled_queue(4, 2, 5, 5, 0, [1, 2, 3, 4])
    spaced = W.regular_arrival_shuffled_queue(4, 2, 5, 5, 10, [1, 2, 3, 4])
    out, skipped = run_batch(K, [burst[0], spaced[0]], [burst[1], spaced[1]], K.POLICY_FCFS, 1)
    assert skipped == 0
    assert out[0][0].tolist() == [0, 1, 2, 3] and out[0][2].tolist() == [10, 20, 30, 40]
    assert out[1][2].tolist() == [10, 10, 10, 10]
    for policy, k in ((K.POLICY_LPM, 1), (K.POLICY_KLPM, 2)):
        out, _ = run_batch(K, [burst[0]], [burst[1]], policy, k)
        assert out[0][0].tolist() == [0, 2, 1, 3] and out[0][2].tolist() == [10, 25, 15, 30]
        assert out[0][1].tolist() == [10, 10, 5, 5]


@pytest.mark.parametrize("policy,k", [(0, 1), (1, 1), (2, 2), (2, 4)])
def test_ten_thousand_regular_arrival_queues_against_the_oracle(K, policy, k):
    """A Monte-Carlo batch over Definition 3: 10,240 queues with random arrival orders and random tie priorities;
    every queue bit-exact with the oracle; the LPM closed form and the k-LPM bound of Theorem 2 hold on the
    device's numbers."""
    rng = np.random.RandomState(100 * policy + k)
    shapes = [(8, 2, 4, 3, 1), (12, 4, 6, 1, 2), (16, 4, 5, 2, 1), (12, 3, 3, 3, 0)]
    queues, arrivals, prios, meta = [], [], [], []
    for q in range(10240):
        n, rep, u, d, s = shapes[q % len(shapes)]
        sigma = (rng.permutation(n) + 1).tolist()
        prompts, arr = W.regular_arrival_shuffled_queue(n, rep, u, d, s, sigma)
        queues.append(prompts); arrivals.append(arr); prios.append(rng.randint(0, 4, size=n).tolist())
        meta.append((n, rep, u, d, s))
    T = 40                                   # >= s n for every shape: everybody has arrived when processing starts
    out, skipped = run_batch(K, queues, arrivals, policy, k, prios, start=T)
    assert skipped == 0
    for q in range(0, 10240):
        want = oracle_queue(queues[q], arrivals[q], policy, k, np.asarray(prios[q], dtype=np.int64), start=T)
        for g, w_ in zip(out[q], want):
            assert np.array_equal(g, w_), q
    for q in range(0, 10240, 7):
        n, rep, u, d, s = meta[q]
        order, unc, ttft, comp = out[q]
        if policy == 1:                      # j-th completion under LPM: T + ceil(j / rep) u + j d
            for pos, j in enumerate(order.tolist(), start=1):
                assert comp[j] == T + math.ceil(pos / rep) * u + d * pos
        if policy == 2 and k == rep:         # Theorem 2's bound for k-LPM with k = the replication factor
            assert ttft.max() <= T + n * (u / k + d - s / k)


@pytest.mark.parametrize("seed", range(3))
def test_ragged_random_queues_with_arrival_gaps_and_c_attn(K, seed):
    """Small-alphabet prompts (long overlaps, empty prompts, identical prompts), queues of 0 .. 70 prompts, idle gaps,
    c_attn = 1/3, and one queue above the size limit that must be left untouched and counted."""
    rng = np.random.RandomState(seed)
    queues, arrivals = [], []
    for q in range(300):
        n = int(rng.randint(0, 71))
        prompts, arr = W.random_small_queue(1000 * seed + q, n, vocab=2, max_len=40, min_len=0, max_gap=30)
        queues.append(prompts); arrivals.append(arr)
    big_n = K.LAST_ONLY_MAX_QUEUE + 1
    queues.insert(17, [[1, 2]] * big_n); arrivals.insert(17, [0] * big_n)
    for policy, k in ((K.POLICY_KLPM, 3), (K.POLICY_LPM, 1), (K.POLICY_FCFS, 1)):
        out, skipped = run_batch(K, queues, arrivals, policy, k, None, 1, 3, 2)
        assert skipped == 1
        assert all((v == -7).all() for v in out[17])
        for q in range(len(queues)):
            if q == 17 or not queues[q]:
                continue
            want = oracle_queue(queues[q], arrivals[q], policy, k, None, 1, 3, 2)
            for g, w_ in zip(out[q], want):
                assert np.array_equal(g, w_), (q, policy)
