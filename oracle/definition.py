"""Definition-level oracle in plain Python, for tiny inputs -- TEST INFRASTRUCTURE ONLY.

Everything is written straight from the paper's definitions with lists and
tuples of ints; no radix tree appears here.  It exists to pin the C++ oracle
(``klpm_oracle.cpp``) to something that is not itself.

  overlap            Section 1.3 (Notation)
  match              max over cached strings of overlap (RadixAttention reuses the
                     longest cached prefix, Section 1)
  completion times   Definition 2
  FCFS / LPM         Section 1;  k-LPM  Algorithm 1
  cache              LAST_ONLY (Definition 2) or TREE = every processed prompt, with
                     LRU eviction of whole leaves under a token budget (Section 1)

The TREE cache is modelled as a *set of strings*: one string per tree node, namely the
full path from the root to the end of that node.  A node's parent is its longest proper
prefix in the set, its edge is what it adds to the parent, and it is a leaf when no other
member extends it.  Nothing is maintained incrementally: parents, leaves and the token
count are recomputed from the set whenever they are needed.
"""
from __future__ import annotations

from fractions import Fraction
from typing import Dict, List, Optional, Sequence, Tuple

FCFS, LPM, KLPM = 0, 1, 2
LAST_ONLY, TREE = 0, 1


def overlap(x: Sequence[int], y: Sequence[int]) -> int:
    n = 0
    while n < len(x) and n < len(y) and x[n] == y[n]:
        n += 1
    return n


class StringSetCache:
    """Prefix cache as a set of node-end strings with per-node last_access."""

    def __init__(self, budget: int = 0):
        self.nodes: Dict[Tuple[int, ...], int] = {}     # node-end string -> last_access
        self.budget = budget
        self.clock = 0
        self.evictions = 0

    def match(self, x: Sequence[int]) -> int:
        return max([overlap(x, s) for s in self.nodes] + [0])

    def match_pos(self, x: Sequence[int]) -> Tuple[int, int, int]:
        """(m, off, depth): the match length, how many tokens of the edge that holds the last matched token
        were matched, and how many tokens lie above that edge.  The edge belongs to the shortest node-end
        string that extends x[:m]; its parent is that string's longest proper prefix in the set."""
        x = tuple(x)
        m = self.match(x)
        if m == 0:
            return 0, 0, 0
        holder = min((s for s in self.nodes if len(s) >= m and s[:m] == x[:m]), key=len)
        depth = len(self.parent(holder))
        return m, m - depth, depth

    def parent(self, s: Tuple[int, ...]) -> Tuple[int, ...]:
        best: Tuple[int, ...] = ()
        for p in self.nodes:
            if len(p) < len(s) and s[:len(p)] == p and len(p) > len(best):
                best = p
        return best

    def tokens(self) -> int:
        return sum(len(s) - len(self.parent(s)) for s in self.nodes)

    def is_leaf(self, s: Tuple[int, ...]) -> bool:
        return not any(len(o) > len(s) and o[:len(s)] == s for o in self.nodes)

    def process(self, x: Sequence[int]) -> int:
        """Charge and store prompt x; returns its uncached token count."""
        x = tuple(x)
        self.clock += 1
        m = self.match(x)
        head = x[:m]
        if m > 0 and head not in self.nodes:
            # boundary at depth m: the node that contains this position is cut in two; the upper
            # part inherits the time stamp of the node it was cut from
            holder = min((s for s in self.nodes if len(s) > m and s[:m] == head), key=len)
            self.nodes[head] = self.nodes[holder]
        for s in list(self.nodes):
            if len(s) <= m and x[:len(s)] == s:
                self.nodes[s] = self.clock             # stamp the path of x
        unc = len(x) - m
        if self.budget > 0:
            while self.tokens() + unc > self.budget:
                leaves = [s for s in self.nodes if self.is_leaf(s)]
                if not leaves:
                    raise RuntimeError("budget")
                victim = min(leaves, key=lambda s: self.nodes[s])
                if self.nodes[victim] >= self.clock:
                    raise RuntimeError("budget")
                del self.nodes[victim]
                self.evictions += 1
        if unc > 0:
            self.nodes[x] = self.clock
        return unc


def schedule(prompts: Sequence[Sequence[int]], arrivals: Sequence[int], policy: int, k: int = 1,
             c_num: int = 0, c_den: int = 1, start_tick: int = 0, cache_mode: int = TREE,
             prefill: Sequence[Sequence[int]] = (), budget: int = 0,
             cache: Optional[StringSetCache] = None, tie_priority: Optional[Sequence[int]] = None,
             score_mode: int = 0):
    """Algorithm 1 / FCFS / LPM with the cost model of Definition 2.
    Returns (order, uncached, ttft, completion); the last three are indexed by query."""
    n = len(prompts)
    if cache_mode == TREE and cache is None:
        cache = StringSetCache(budget)
        for p in prefill:
            cache.process(p)
    last: Optional[Sequence[int]] = None

    def match(x):
        if cache_mode == LAST_ONLY:
            return 0 if last is None else overlap(x, last)
        return cache.match(x)

    done = [False] * n
    order: List[int] = []
    unc = [0] * n
    ttft = [0] * n
    comp = [0] * n
    now = start_tick
    for c in range(n):
        waiting = [i for i in range(n) if not done[i] and arrivals[i] <= now]
        if not waiting:
            now = min(arrivals[i] for i in range(n) if not done[i])
            waiting = [i for i in range(n) if not done[i] and arrivals[i] <= now]
        if policy == FCFS or (policy == KLPM and c % k == 0):
            j = min(waiting, key=lambda i: (arrivals[i], i))
        else:
            def score(i):
                mi = match(prompts[i])
                if score_mode == 1:         # the prompt's hit rate, an exact rational (0 for an empty prompt)
                    return Fraction(mi, len(prompts[i])) if len(prompts[i]) else Fraction(0)
                return mi
            j = min(waiting, key=lambda i: (-score(i), tie_priority[i] if tie_priority is not None else 0, arrivals[i], i))
        x = prompts[j]
        if cache_mode == LAST_ONLY:
            u = len(x) - match(x)
            last = x
        else:
            u = cache.process(x)
        begin = max(now, arrivals[j])
        R = begin + (c_den + c_num * len(x)) * u
        order.append(j)
        unc[j], ttft[j], comp[j] = u, R - arrivals[j], R
        done[j] = True
        now = R
    return order, unc, ttft, comp


def select(match_len: Sequence[int], arrivals: Sequence[int], waiting: Sequence[int], pick_counter: int, policy: int, k: int = 1) -> int:
    """One decision of Algorithm 1 over a snapshot: the rule of schedule() above, on given match lengths."""
    idx = [i for i in range(len(match_len)) if waiting[i]]
    if not idx:
        return -1
    if policy == FCFS or (policy == KLPM and pick_counter % k == 0):
        return min(idx, key=lambda i: (arrivals[i], i))
    return min(idx, key=lambda i: (-match_len[i], arrivals[i], i))


def replay(order: Sequence[int], prompts, arrivals, c_num: int = 0, c_den: int = 1, start_tick: int = 0,
           cache_mode: int = TREE, prefill=(), budget: int = 0):
    """Definition 2 along a fixed order.  Returns (uncached, ttft, completion) indexed by query."""
    n = len(prompts)
    cache = StringSetCache(budget)
    for p in prefill:
        cache.process(p)
    last = None
    unc, ttft, comp = [0] * n, [0] * n, [0] * n
    now = start_tick
    for j in order:
        x = prompts[j]
        if cache_mode == LAST_ONLY:
            u = len(x) - (0 if last is None else overlap(x, last))
            last = x
        else:
            u = cache.process(x)
        R = max(now, arrivals[j]) + (c_den + c_num * len(x)) * u
        unc[j], ttft[j], comp[j] = u, R - arrivals[j], R
        now = R
    return unc, ttft, comp
