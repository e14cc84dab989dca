"""ctypes binding of libklpm.so: argument marshalling only.

Same names as the C ABI (include/klpm.h).  Tensors must live on the CUDA device; every step of the
path runs in the library's kernels.  There is no CPU fallback: importing this module fails if the
library has not been built, and every call fails on a non-CUDA tensor.
"""
from __future__ import annotations

import ctypes
import os
from typing import Optional

import torch

_HERE = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.environ.get("KLPM_LIB") or os.path.join(_HERE, "libklpm.so")

RT_OK, RT_ERR_INVALID, RT_ERR_CAPACITY, RT_ERR_BUDGET, RT_ERR_LIMIT, RT_ERR_CUDA = 0, -1, -2, -3, -4, -5
RT_ERR_TOO_LARGE = -6
SELECT_NOALLOC_MAX_QUERIES = 1 << 22
POLICY_FCFS, POLICY_LPM, POLICY_KLPM = 0, 1, 2
_ERR = {-1: "RT_ERR_INVALID", -2: "RT_ERR_CAPACITY", -3: "RT_ERR_BUDGET", -4: "RT_ERR_LIMIT", -5: "RT_ERR_CUDA",
        -6: "RT_ERR_TOO_LARGE"}


class KlpmError(RuntimeError):
    def __init__(self, code: int, where: str):
        super().__init__("%s returned %s (%d)" % (where, _ERR.get(code, "?"), code))
        self.code = code


class rt_config(ctypes.Structure):
    _fields_ = [("vocab", ctypes.c_int32), ("max_nodes", ctypes.c_int64), ("max_pool_tokens", ctypes.c_int64),
                ("budget_tokens", ctypes.c_int64), ("max_clock", ctypes.c_int64)]


class klpm_params(ctypes.Structure):
    _fields_ = [("policy", ctypes.c_int32), ("k", ctypes.c_int32), ("c_num", ctypes.c_int64),
                ("c_den", ctypes.c_int64), ("start_tick", ctypes.c_int64)]


if not os.path.exists(LIB_PATH):
    raise ImportError("libklpm.so is not built: run `python -m paper_2502_04677_b200.build` "
                      "(there is no CPU fallback for this library)")

_lib = ctypes.CDLL(LIB_PATH)
_vp, _i32, _i64 = ctypes.c_void_p, ctypes.c_int32, ctypes.c_int64

_lib.klpm_abi_version.restype = _i32
_lib.rt_create.restype = _i32
_lib.rt_create.argtypes = [ctypes.POINTER(rt_config), ctypes.POINTER(_vp)]
_lib.rt_build.restype = _i32
_lib.rt_build.argtypes = [_vp, _vp, _i32, ctypes.POINTER(rt_config), _vp, ctypes.POINTER(_vp)]
_lib.rt_insert.restype = _i32
_lib.rt_insert.argtypes = [_vp, _vp, _vp, _i32, _vp, _vp]
_lib.rt_match_batch.restype = _i32
_lib.rt_match_batch.argtypes = [_vp, _vp, _vp, _i32, _vp, _vp, _vp, _vp]
_lib.rt_match_batch_ex.restype = _i32
_lib.rt_match_batch_ex.argtypes = [_vp, _vp, _vp, _i32, _vp, _vp, _vp, _vp, _vp]
_lib.rt_stats.restype = _i32
_lib.rt_stats.argtypes = [_vp] + [ctypes.POINTER(_i64)] * 5
_lib.rt_clone.restype = _i32
_lib.rt_clone.argtypes = [_vp, _vp, ctypes.POINTER(_vp)]
_lib.rt_checkpoint.restype = _i32
_lib.rt_checkpoint.argtypes = [_vp, _vp]
_lib.rt_rollback.restype = _i32
_lib.rt_rollback.argtypes = [_vp, _vp]
_lib.rt_status_detail.restype = _i32
_lib.rt_status_detail.argtypes = [_vp, ctypes.POINTER(_i32)]
_lib.rt_sync_status.restype = _i32
_lib.rt_sync_status.argtypes = [_vp, _vp]
_lib.rt_destroy.restype = _i32
_lib.rt_destroy.argtypes = [_vp]
_lib.klpm_select.restype = _i32
_lib.klpm_select.argtypes = [_vp, _vp, _vp, _i32, _i64, ctypes.POINTER(klpm_params), _vp, _vp]
_lib.klpm_select_topk.restype = _i32
_lib.klpm_select_topk.argtypes = [_vp, _vp, _vp, _i32, _i32, _vp, _vp]
_lib.klpm_select_noalloc.restype = _i32
_lib.klpm_select_noalloc.argtypes = [_vp, _vp, _vp, _i32, _i64, ctypes.POINTER(klpm_params), _vp, _vp]
_lib.klpm_replay.restype = _i32
_lib.klpm_replay.argtypes = [_vp, _vp, _i32, _vp, _vp, _vp, _i32, ctypes.POINTER(klpm_params), _vp, _vp, _vp, _vp]
_lib.klpm_run_ex.restype = _i32
_lib.klpm_run_ex.argtypes = [_vp, _vp, _vp, _vp, _i32, ctypes.POINTER(klpm_params), _vp, _i32, _vp, _vp, _vp, _vp, _vp, _vp]
_lib.klpm_batch_times.restype = _i32
_lib.klpm_batch_times.argtypes = [_vp, _i32, _vp, _vp, _i32, _i32, _vp, _vp, _vp, _vp]
_lib.klpm_run_last_only_batch.restype = _i32
_lib.klpm_run_last_only_batch.argtypes = [_vp, _vp, _vp, _vp, _vp, _i32, ctypes.POINTER(klpm_params), _vp, _vp, _vp, _vp, _vp, _vp]
_lib.rt_debug_counters.restype = _i32
_lib.rt_debug_counters.argtypes = [_vp, ctypes.POINTER(_i64 * 16)]
_lib.klpm_debug_set.restype = _i32
_lib.klpm_debug_set.argtypes = [ctypes.c_char_p, _i64]
_lib.klpm_run_path.restype = _i32
_lib.klpm_run_path.argtypes = [_vp]
_lib.klpm_run.restype = _i32
_lib.klpm_run.argtypes = [_vp, _vp, _vp, _vp, _i32, ctypes.POINTER(klpm_params), _vp, _vp, _vp, _vp, _vp]

MATCH_STATE_BYTES = 32

EXPORTS = ["klpm_abi_version", "rt_create", "rt_build", "rt_insert", "rt_match_batch", "rt_match_batch_ex", "rt_stats",
           "rt_sync_status", "rt_status_detail", "rt_clone", "rt_checkpoint", "rt_rollback", "rt_destroy", "klpm_select", "klpm_select_topk", "klpm_select_noalloc", "klpm_replay", "klpm_run", "klpm_run_ex", "klpm_run_path", "klpm_batch_times", "klpm_debug_set", "klpm_run_last_only_batch", "rt_debug_counters"]


def lib() -> ctypes.CDLL:
    return _lib


def _dev(t: Optional[torch.Tensor], dtype, name: str, nullable: bool = False):
    if t is None:
        if nullable:
            return None
        raise ValueError("%s must not be None" % name)
    if not t.is_cuda:
        raise ValueError("%s must be a CUDA tensor (this library has no CPU path)" % name)
    if t.dtype != dtype or not t.is_contiguous():
        raise ValueError("%s must be a contiguous %s tensor" % (name, dtype))
    return ctypes.c_void_p(t.data_ptr())


def _stream() -> ctypes.c_void_p:
    return ctypes.c_void_p(torch.cuda.current_stream().cuda_stream)


def _check(code: int, where: str) -> None:
    if code != RT_OK:
        raise KlpmError(code, where)


def make_params(policy: int, k: int = 1, c_num: int = 0, c_den: int = 1, start_tick: int = 0) -> klpm_params:
    return klpm_params(int(policy), int(k), int(c_num), int(c_den), int(start_tick))


class Tree:
    """Handle of a device radix tree (rt_tree*)."""

    def __init__(self, handle: ctypes.c_void_p):
        self._h = handle

    @property
    def handle(self) -> ctypes.c_void_p:
        if not self._h:
            raise ValueError("tree was destroyed")
        return self._h

    def destroy(self) -> None:
        if self._h:
            _check(_lib.rt_destroy(self._h), "rt_destroy")
            self._h = None

    def __del__(self):
        try:
            self.destroy()
        except Exception:
            pass


def rt_create(max_nodes: int, max_pool_tokens: int, budget_tokens: int = 0, vocab: int = 0, max_clock: int = 0) -> Tree:
    cfg = rt_config(int(vocab), int(max_nodes), int(max_pool_tokens), int(budget_tokens), int(max_clock))
    h = ctypes.c_void_p()
    _check(_lib.rt_create(ctypes.byref(cfg), ctypes.byref(h)), "rt_create")
    return Tree(h)


def rt_build(tokens: torch.Tensor, offsets: torch.Tensor, max_nodes: int, max_pool_tokens: int,
             budget_tokens: int = 0, vocab: int = 0, max_clock: int = 0) -> Tree:
    cfg = rt_config(int(vocab), int(max_nodes), int(max_pool_tokens), int(budget_tokens), int(max_clock))
    h = ctypes.c_void_p()
    n = offsets.numel() - 1
    _check(_lib.rt_build(_dev(tokens, torch.int32, "tokens", n == 0), _dev(offsets, torch.int64, "offsets"), n,
                         ctypes.byref(cfg), _stream(), ctypes.byref(h)), "rt_build")
    return Tree(h)


def rt_insert(tree: Tree, tokens: torch.Tensor, offsets: torch.Tensor, new_tokens: Optional[torch.Tensor] = None) -> None:
    n = offsets.numel() - 1
    _check(_lib.rt_insert(tree.handle, _dev(tokens, torch.int32, "tokens"), _dev(offsets, torch.int64, "offsets"), n,
                          _dev(new_tokens, torch.int32, "new_tokens", True), _stream()), "rt_insert")


def rt_match_batch(tree: Tree, q_tokens: torch.Tensor, q_offsets: torch.Tensor, match_len: torch.Tensor,
                   term_node: Optional[torch.Tensor] = None, term_off: Optional[torch.Tensor] = None) -> None:
    nq = q_offsets.numel() - 1
    _check(_lib.rt_match_batch(tree.handle, _dev(q_tokens, torch.int32, "q_tokens"), _dev(q_offsets, torch.int64, "q_offsets"),
                               nq, _dev(match_len, torch.int32, "match_len"), _dev(term_node, torch.int32, "term_node", True),
                               _dev(term_off, torch.int32, "term_off", True), _stream()), "rt_match_batch")


def match_state_buffer(nq: int, device) -> torch.Tensor:
    """Device memory for the records rt_match_batch_ex keeps for klpm_run_ex (klpm_match_state[nq], opaque)."""
    return torch.empty((max(int(nq), 1), MATCH_STATE_BYTES // 8), dtype=torch.int64, device=device)


def rt_match_batch_ex(tree: Tree, q_tokens: torch.Tensor, q_offsets: torch.Tensor, match_len: torch.Tensor,
                      term_node: Optional[torch.Tensor] = None, term_off: Optional[torch.Tensor] = None,
                      state: Optional[torch.Tensor] = None) -> None:
    nq = q_offsets.numel() - 1
    if state is not None and state.numel() * 8 < nq * MATCH_STATE_BYTES:
        raise ValueError("state must hold %d bytes per query" % MATCH_STATE_BYTES)
    _check(_lib.rt_match_batch_ex(tree.handle, _dev(q_tokens, torch.int32, "q_tokens"), _dev(q_offsets, torch.int64, "q_offsets"),
                                  nq, _dev(match_len, torch.int32, "match_len"), _dev(term_node, torch.int32, "term_node", True),
                                  _dev(term_off, torch.int32, "term_off", True), _dev(state, torch.int64, "state", True),
                                  _stream()), "rt_match_batch_ex")


def rt_stats(tree: Tree) -> dict:
    v = [ctypes.c_int64() for _ in range(5)]
    _check(_lib.rt_stats(tree.handle, *[ctypes.byref(x) for x in v]), "rt_stats")
    return dict(n_nodes=v[0].value, tokens=v[1].value, clock=v[2].value, evictions=v[3].value, pool_used=v[4].value)


def rt_clone(tree: Tree) -> Tree:
    h = ctypes.c_void_p()
    _check(_lib.rt_clone(tree.handle, _stream(), ctypes.byref(h)), "rt_clone")
    return Tree(h)


def rt_checkpoint(tree: Tree) -> None:
    _check(_lib.rt_checkpoint(tree.handle, _stream()), "rt_checkpoint")


def rt_rollback(tree: Tree) -> None:
    _check(_lib.rt_rollback(tree.handle, _stream()), "rt_rollback")


def rt_status_detail(tree: Tree) -> int:
    d = ctypes.c_int32()
    _check(_lib.rt_status_detail(tree.handle, ctypes.byref(d)), "rt_status_detail")
    return int(d.value)


def rt_sync_status(tree: Tree) -> int:
    return int(_lib.rt_sync_status(tree.handle, _stream()))


def rt_destroy(tree: Tree) -> None:
    tree.destroy()


def _same_length(match_len: torch.Tensor, arrival: torch.Tensor, waiting: torch.Tensor) -> int:
    n = match_len.numel()
    if arrival.numel() != n or waiting.numel() != n:
        raise ValueError("match_len, arrival and waiting must have the same number of elements")
    return n


def klpm_select(match_len: torch.Tensor, arrival: torch.Tensor, waiting: torch.Tensor, pick_counter: int,
                params: klpm_params, pick: torch.Tensor) -> None:
    _same_length(match_len, arrival, waiting)
    _check(_lib.klpm_select(_dev(match_len, torch.int32, "match_len"), _dev(arrival, torch.int64, "arrival"),
                            _dev(waiting, torch.uint8, "waiting"), match_len.numel(), int(pick_counter),
                            ctypes.byref(params), _dev(pick, torch.int32, "pick"), _stream()), "klpm_select")


def klpm_select_topk(match_len: torch.Tensor, arrival: torch.Tensor, waiting: torch.Tensor, out: torch.Tensor) -> None:
    """out (int32[kk]) receives the kk best longest-match candidates of this snapshot, best first."""
    _same_length(match_len, arrival, waiting)
    _check(_lib.klpm_select_topk(_dev(match_len, torch.int32, "match_len"), _dev(arrival, torch.int64, "arrival"),
                                 _dev(waiting, torch.uint8, "waiting"), match_len.numel(), out.numel(),
                                 _dev(out, torch.int32, "out"), _stream()), "klpm_select_topk")


def klpm_select_noalloc(match_len: torch.Tensor, arrival: torch.Tensor, waiting: torch.Tensor, pick_counter: int,
                        params: klpm_params, pick: torch.Tensor) -> None:
    """klpm_select without any device allocation inside the library (fixed scratch; at most
    SELECT_NOALLOC_MAX_QUERIES queries; calls must not overlap on the GPU)."""
    n = _same_length(match_len, arrival, waiting)
    _check(_lib.klpm_select_noalloc(_dev(match_len, torch.int32, "match_len"), _dev(arrival, torch.int64, "arrival"),
                                    _dev(waiting, torch.uint8, "waiting"), n, int(pick_counter),
                                    ctypes.byref(params), _dev(pick, torch.int32, "pick"), _stream()),
           "klpm_select_noalloc")


def klpm_replay(tree: Tree, order: torch.Tensor, q_tokens: torch.Tensor, q_offsets: torch.Tensor, arrival: torch.Tensor,
                params: klpm_params, uncached: torch.Tensor, ttft: torch.Tensor,
                completion: Optional[torch.Tensor] = None) -> None:
    _check(_lib.klpm_replay(tree.handle, _dev(order, torch.int32, "order"), order.numel(),
                            _dev(q_tokens, torch.int32, "q_tokens"), _dev(q_offsets, torch.int64, "q_offsets"),
                            _dev(arrival, torch.int64, "arrival"), arrival.numel(), ctypes.byref(params),
                            _dev(uncached, torch.int32, "uncached"), _dev(ttft, torch.int64, "ttft"),
                            _dev(completion, torch.int64, "completion", True), _stream()), "klpm_replay")


def klpm_run(tree: Tree, q_tokens: torch.Tensor, q_offsets: torch.Tensor, arrival: torch.Tensor, params: klpm_params,
             order: torch.Tensor, uncached: torch.Tensor, ttft: torch.Tensor,
             completion: Optional[torch.Tensor] = None) -> None:
    n = arrival.numel()
    _check(_lib.klpm_run(tree.handle, _dev(q_tokens, torch.int32, "q_tokens"), _dev(q_offsets, torch.int64, "q_offsets"),
                         _dev(arrival, torch.int64, "arrival"), n, ctypes.byref(params), _dev(order, torch.int32, "order"),
                         _dev(uncached, torch.int32, "uncached"), _dev(ttft, torch.int64, "ttft"),
                         _dev(completion, torch.int64, "completion", True), _stream()), "klpm_run")


RUN_PATH_NONE, RUN_PATH_ONE_BY_ONE, RUN_PATH_GROUPED = 0, 1, 2


def klpm_run_path(tree: Tree) -> int:
    """Which loop the last klpm_run / klpm_run_ex on this tree took (RUN_PATH_*)."""
    return int(_lib.klpm_run_path(tree.handle))


def klpm_batch_times(order: torch.Tensor, arrival: torch.Tensor, completion: torch.Tensor, batch_size: int,
                     ttft_b: torch.Tensor, completion_b: torch.Tensor, n_skipped: Optional[torch.Tensor] = None) -> None:
    n = arrival.numel()
    if completion.numel() != n or ttft_b.numel() != n or completion_b.numel() != n:
        raise ValueError("arrival, completion, ttft_b and completion_b must have one entry per query")
    _check(_lib.klpm_batch_times(_dev(order, torch.int32, "order"), order.numel(), _dev(arrival, torch.int64, "arrival"),
                                 _dev(completion, torch.int64, "completion"), n, int(batch_size),
                                 _dev(ttft_b, torch.int64, "ttft_b"), _dev(completion_b, torch.int64, "completion_b"),
                                 _dev(n_skipped, torch.int32, "n_skipped", True), _stream()), "klpm_batch_times")


LAST_ONLY_MAX_QUEUE = 1024


def klpm_run_last_only_batch(tokens: torch.Tensor, offsets: torch.Tensor, arrival: torch.Tensor,
                             tie_priority: Optional[torch.Tensor], queue_offsets: torch.Tensor, params: klpm_params,
                             order: torch.Tensor, uncached: torch.Tensor, ttft: torch.Tensor,
                             completion: Optional[torch.Tensor] = None, n_skipped: Optional[torch.Tensor] = None) -> None:
    """Many independent queues under the last-prompt cache, one warp each (see include/klpm.h)."""
    n_prompts = offsets.numel() - 1
    for t, name in ((arrival, "arrival"), (order, "order"), (uncached, "uncached"), (ttft, "ttft")):
        if t.numel() != n_prompts:
            raise ValueError("%s must have one entry per prompt" % name)
    _check(_lib.klpm_run_last_only_batch(_dev(tokens, torch.int32, "tokens"), _dev(offsets, torch.int64, "offsets"),
                                         _dev(arrival, torch.int64, "arrival"),
                                         _dev(tie_priority, torch.int64, "tie_priority", True),
                                         _dev(queue_offsets, torch.int32, "queue_offsets"), queue_offsets.numel() - 1,
                                         ctypes.byref(params), _dev(order, torch.int32, "order"),
                                         _dev(uncached, torch.int32, "uncached"), _dev(ttft, torch.int64, "ttft"),
                                         _dev(completion, torch.int64, "completion", True),
                                         _dev(n_skipped, torch.int32, "n_skipped", True), _stream()),
           "klpm_run_last_only_batch")


def rt_debug_counters(tree: Tree) -> dict:
    """What the grouped loop of the last klpm_run on this tree did (see include/klpm.h)."""
    v = (_i64 * 16)()
    _check(_lib.rt_debug_counters(tree.handle, ctypes.byref(v)), "rt_debug_counters")
    names = ("careful_steps", "cta_dissolves", "fallback_scans", "fallen_back", "evictions", "cycles_tree", "cycles_scans",
             "cycles_cta_dissolves", "cta_batches_tried", "cta_batches", "cta_batch_decisions", "warp_steps",
             "warp_step_decisions", "single_decisions", "cycles_cta_batches", "cycles_warp_steps")
    return dict(zip(names, [int(x) for x in v]))


def klpm_debug_set(name: str, value: int) -> None:
    """Process-wide test/debug settings of the library (see include/klpm.h); value < 0 restores the default."""
    _check(_lib.klpm_debug_set(name.encode(), int(value)), "klpm_debug_set")


def klpm_run_ex(tree: Tree, q_tokens: torch.Tensor, q_offsets: torch.Tensor, arrival: torch.Tensor, params: klpm_params,
                tie_priority: Optional[torch.Tensor], score_mode: int, order: torch.Tensor, uncached: torch.Tensor,
                ttft: torch.Tensor, completion: Optional[torch.Tensor] = None,
                match_state: Optional[torch.Tensor] = None) -> None:
    n = arrival.numel()
    _check(_lib.klpm_run_ex(tree.handle, _dev(q_tokens, torch.int32, "q_tokens"), _dev(q_offsets, torch.int64, "q_offsets"),
                            _dev(arrival, torch.int64, "arrival"), n, ctypes.byref(params),
                            _dev(tie_priority, torch.int64, "tie_priority", True), int(score_mode),
                            _dev(match_state, torch.int64, "match_state", True),
                            _dev(order, torch.int32, "order"), _dev(uncached, torch.int32, "uncached"),
                            _dev(ttft, torch.int64, "ttft"), _dev(completion, torch.int64, "completion", True), _stream()),
           "klpm_run_ex")
