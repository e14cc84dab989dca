"""CPU oracle for the k-LPM scheduling path -- TEST INFRASTRUCTURE ONLY.

Python face of ``klpm_oracle.cpp`` (a plain pointer-based radix tree, the
scheduling policies and the cost model, written from the paper) plus
``definition.py`` (the same things written straight from the definitions with
Python lists, for tiny inputs).  Nothing here is used by the CUDA library or
its binding; only tests, the smoke check and the benchmark's CPU baseline
import this package.
"""
from __future__ import annotations

import ctypes
import os
import subprocess
from typing import Optional, Sequence, Tuple

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "klpm_oracle.cpp")
_LIB = os.path.join(_HERE, "libklpm_oracle.so")

POLICY_FCFS, POLICY_LPM, POLICY_KLPM = 0, 1, 2
CACHE_LAST_ONLY, CACHE_TREE = 0, 1
TIER_REMATCH, TIER_UPDATE = 1, 2


def build(force: bool = False) -> str:
    """Compile the oracle with g++ (no CUDA involved)."""
    if force or not os.path.exists(_LIB) or os.path.getmtime(_LIB) < os.path.getmtime(_SRC):
        tmp = _LIB + ".%d.tmp" % os.getpid()
        subprocess.check_call(["g++", "-O2", "-std=c++17", "-fPIC", "-shared", "-pthread", _SRC, "-o", tmp])
        os.replace(tmp, _LIB)
    return _LIB


_lib = None


def lib():
    global _lib
    if _lib is None:
        L = ctypes.CDLL(build())
        vp, i32, i64 = ctypes.c_void_p, ctypes.c_int32, ctypes.c_int64
        L.oc_overlap.restype = i64
        L.oc_overlap.argtypes = [vp, i64, vp, i64]
        L.oc_match_bruteforce.restype = None
        L.oc_match_bruteforce.argtypes = [vp, vp, i32, vp, vp, i32, vp]
        L.oc_tree_new.restype = vp
        L.oc_tree_new.argtypes = [i64, i32]
        L.oc_tree_free.restype = None
        L.oc_tree_free.argtypes = [vp]
        L.oc_tree_stats.restype = None
        L.oc_tree_stats.argtypes = [vp, vp, vp, vp, vp]
        L.oc_tree_insert.restype = i32
        L.oc_tree_insert.argtypes = [vp, vp, vp, i32, vp]
        L.oc_tree_match.restype = None
        L.oc_tree_match.argtypes = [vp, vp, vp, i32, vp, i32]
        L.oc_tree_match_pos.restype = None
        L.oc_tree_match_pos.argtypes = [vp, vp, vp, i32, vp, vp, vp]
        L.oc_select.restype = i32
        L.oc_select.argtypes = [vp, vp, vp, i32, i64, i32, i32]
        L.oc_replay.restype = i32
        L.oc_replay.argtypes = [vp, vp, i32, vp, vp, vp, i32, i64, i64, i64, i32, vp, vp, vp]
        L.oc_batch_times.restype = None
        L.oc_batch_times.argtypes = [vp, i32, vp, vp, i32, vp, vp]
        L.oc_schedule_ex.restype = i32
        L.oc_schedule_ex.argtypes = [vp, vp, vp, vp, i32, i32, i32, i64, i64, i64, i32, i32, vp, i32, vp, vp, vp, vp]
        L.oc_schedule.restype = i32
        L.oc_schedule.argtypes = [vp, vp, vp, vp, i32, i32, i32, i64, i64, i64, i32, i32, vp, vp, vp, vp]
        _lib = L
    return _lib


def _i32(a) -> np.ndarray:
    return np.ascontiguousarray(np.asarray(a), dtype=np.int32)


def _i64(a) -> np.ndarray:
    return np.ascontiguousarray(np.asarray(a), dtype=np.int64)


def _p(a: Optional[np.ndarray]):
    return None if a is None else a.ctypes.data_as(ctypes.c_void_p)


def overlap(x: Sequence[int], y: Sequence[int]) -> int:
    x, y = _i32(x), _i32(y)
    return int(lib().oc_overlap(_p(x), len(x), _p(y), len(y)))


def match_bruteforce(q_tokens, q_offsets, c_tokens, c_offsets, match_len: Optional[np.ndarray] = None) -> np.ndarray:
    """max over cached prompts y of overlap(q, y); accumulates into match_len if given."""
    qt, qo, ct, co = _i32(q_tokens), _i64(q_offsets), _i32(c_tokens), _i64(c_offsets)
    out = np.zeros(len(qo) - 1, dtype=np.int32) if match_len is None else match_len
    lib().oc_match_bruteforce(_p(qt), _p(qo), len(qo) - 1, _p(ct), _p(co), len(co) - 1, _p(out))
    return out


class OracleTree:
    """Radix tree of processed prompts with LRU eviction (TREE cache mode)."""

    def __init__(self, budget_tokens: int = 0, indexed: bool = True):
        self._h = lib().oc_tree_new(int(budget_tokens), 1 if indexed else 0)

    def close(self):
        if self._h:
            lib().oc_tree_free(self._h)
            self._h = None

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass

    def insert(self, tokens, offsets) -> np.ndarray:
        t, o = _i32(tokens), _i64(offsets)
        new = np.zeros(len(o) - 1, dtype=np.int32)
        rc = lib().oc_tree_insert(self._h, _p(t), _p(o), len(o) - 1, _p(new))
        if rc:
            raise RuntimeError("oracle: budget cannot hold the prompt (%d)" % rc)
        return new

    def match(self, tokens, offsets, threads: int = 1) -> np.ndarray:
        t, o = _i32(tokens), _i64(offsets)
        out = np.zeros(len(o) - 1, dtype=np.int32)
        lib().oc_tree_match(self._h, _p(t), _p(o), len(o) - 1, _p(out), threads)
        return out

    def match_pos(self, tokens, offsets) -> Tuple[np.ndarray, np.ndarray, np.ndarray]:
        """match() plus where each match ended: (match_len, term_off, term_depth) -- how many tokens of the edge
        holding the last matched token were matched, and how many tokens lie on the path above that edge."""
        t, o = _i32(tokens), _i64(offsets)
        n = len(o) - 1
        m, off, depth = (np.zeros(n, dtype=np.int32) for _ in range(3))
        lib().oc_tree_match_pos(self._h, _p(t), _p(o), n, _p(m), _p(off), _p(depth))
        return m, off, depth

    def stats(self) -> dict:
        v = [ctypes.c_int64() for _ in range(4)]
        lib().oc_tree_stats(self._h, *[ctypes.byref(x) for x in v])
        return dict(n_nodes=v[0].value, tokens=v[1].value, clock=v[2].value, evictions=v[3].value)


def schedule(tokens, offsets, arrivals, policy: int, k: int = 1, c_num: int = 0, c_den: int = 1,
             start_tick: int = 0, cache_mode: int = CACHE_TREE, tier: int = TIER_UPDATE,
             tree: Optional[OracleTree] = None, tie_priority=None, score_mode: int = 0
             ) -> Tuple[np.ndarray, np.ndarray, np.ndarray, np.ndarray]:
    """Run FCFS / LPM / k-LPM over the stream.  Returns order, uncached, ttft, completion.
    tie_priority (optional int64 per query): smaller wins among equal scores of a longest-match pick.
    score_mode 1: the score is the hit rate match / length (an exact rational) instead of the match length."""
    t, o, a = _i32(tokens), _i64(offsets), _i64(arrivals)
    n = len(o) - 1
    if cache_mode == CACHE_TREE and tree is None:
        tree = OracleTree()
    order = np.zeros(n, dtype=np.int32)
    unc = np.zeros(n, dtype=np.int32)
    ttft = np.zeros(n, dtype=np.int64)
    comp = np.zeros(n, dtype=np.int64)
    pr = None if tie_priority is None else _i64(tie_priority)
    rc = lib().oc_schedule_ex(tree._h if tree is not None else None, _p(t), _p(o), _p(a), n, policy, max(1, int(k)),
                              c_num, c_den, start_tick, cache_mode, tier, _p(pr), int(score_mode),
                              _p(order), _p(unc), _p(ttft), _p(comp))
    if rc:
        raise RuntimeError("oracle: schedule failed (%d)" % rc)
    return order, unc, ttft, comp


def select(match_len, arrivals, waiting, pick_counter: int, policy: int, k: int = 1) -> int:
    """One decision of Algorithm 1 over a snapshot of the queue: index of the pick, -1 if nobody is waiting."""
    m, a = _i32(match_len), _i64(arrivals)
    w = np.ascontiguousarray(np.asarray(waiting), dtype=np.uint8)
    return int(lib().oc_select(_p(m), _p(a), _p(w), len(m), int(pick_counter), int(policy), max(1, int(k))))


def replay(order, tokens, offsets, arrivals, c_num: int = 0, c_den: int = 1, start_tick: int = 0,
           cache_mode: int = CACHE_TREE, tree: Optional[OracleTree] = None):
    """Definition 2 along a fixed processing order.  Returns uncached, ttft, completion (indexed by query)."""
    od, t, o, a = _i32(order), _i32(tokens), _i64(offsets), _i64(arrivals)
    n = len(o) - 1
    if cache_mode == CACHE_TREE and tree is None:
        tree = OracleTree()
    unc = np.zeros(n, dtype=np.int32)
    ttft = np.zeros(n, dtype=np.int64)
    comp = np.zeros(n, dtype=np.int64)
    rc = lib().oc_replay(tree._h if tree is not None else None, _p(od), len(od), _p(t), _p(o), _p(a), n,
                         c_num, c_den, start_tick, cache_mode, _p(unc), _p(ttft), _p(comp))
    if rc:
        raise RuntimeError("oracle: replay failed (%d)" % rc)
    return unc, ttft, comp


def batch_times(order, arrivals, completion, B: int):
    """Section 2.1: with batch size B a query finishes with the last query of its bin of the order.
    Returns ttft_b, completion_b (indexed by query)."""
    od, a, c = _i32(order), _i64(arrivals), _i64(completion)
    ttft = np.zeros(len(a), dtype=np.int64)
    comp = np.zeros(len(a), dtype=np.int64)
    lib().oc_batch_times(_p(od), len(od), _p(a), _p(c), int(B), _p(ttft), _p(comp))
    return ttft, comp
