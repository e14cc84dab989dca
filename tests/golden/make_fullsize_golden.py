#!/usr/bin/env python
"""Writes tests/golden/fullsize_<config>.json: what the CPU oracle computes on a configuration at its full size.

Calls only the input generators and `oracle/`.  For the chosen configuration it builds the oracle's radix
tree from the cached prompts (in chunks), matches every query, runs the scheduling loop for the k values
the configuration names (oracle tier UPDATE), and stores SHA-256 digests of the complete output arrays
(little-endian int32 / int64, indexed as the C ABI documents) plus a sample of the values themselves.
The GPU tests recompute the same digests from the CUDA library's outputs.

    python tests/golden/make_fullsize_golden.py medium [--scale 1.0] [--no-schedule]

Takes minutes (adversarial: generating 16.6 G prompt tokens on the CPU dominates).
"""
from __future__ import annotations

import argparse
import hashlib
import json
import os
import sys
import time

import numpy as np
import torch

ROOT = os.path.dirname(os.path.dirname(os.path.dirname(os.path.abspath(__file__))))
sys.path.insert(0, ROOT)

import oracle  # noqa: E402
from paper_2502_04677_b200 import workloads as W  # noqa: E402


def digest(a: np.ndarray) -> str:
    return hashlib.sha256(np.ascontiguousarray(a).tobytes()).hexdigest()


def build_tree(w: W.Workload, chunk_tokens: int = 1 << 28) -> oracle.OracleTree:
    tree = oracle.OracleTree(w.budget_tokens)
    off_all = w.prefill.offsets()
    a, n = 0, w.prefill.n
    while a < n:
        limit = int(off_all[a]) + chunk_tokens
        b = int(torch.searchsorted(off_all, torch.tensor(limit), right=True)) - 1
        b = max(a + 1, min(b, n))
        tok, off = w.prefill.materialize("cpu", a, b)
        tree.insert(tok.numpy(), off.numpy())
        a = b
    return tree


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("config", choices=sorted(W.WORKLOADS))
    ap.add_argument("--scale", type=float, default=1.0)
    ap.add_argument("--no-schedule", action="store_true")
    ap.add_argument("--threads", type=int, default=os.cpu_count() or 1)
    args = ap.parse_args()
    name = args.config
    w = W.WORKLOADS[name]() if name == "tiny" else W.WORKLOADS[name](scale=args.scale)
    out = {"config": name, "scale": args.scale if name != "tiny" else 1.0, "recipe": w.recipe,
           "queries": w.queries.n, "prefill": w.prefill.n, "budget_tokens": w.budget_tokens,
           "written_by": "tests/golden/make_fullsize_golden.py (oracle only)"}
    fname = "fullsize_%s.json" % name if (name == "tiny" or args.scale == 1.0) else "scale%g_%s.json" % (args.scale, name)
    path = os.path.join(os.path.dirname(os.path.abspath(__file__)), fname)
    t0 = time.time()
    tree = build_tree(w)
    out["tree"] = tree.stats()
    print("tree built in %.0f s: %s" % (time.time() - t0, out["tree"]), flush=True)
    qt, qo = w.queries.materialize()
    qtn, qon = qt.numpy(), qo.numpy()
    t0 = time.time()
    m = tree.match(qtn, qon, threads=args.threads)
    print("matched in %.1f s" % (time.time() - t0), flush=True)
    step = max(1, w.queries.n // 257)
    out["match_len"] = {"sha256": digest(m.astype("<i4")), "sum": int(m.astype(np.int64).sum()),
                        "sample_step": step, "sample": m[::step].tolist()}
    if not args.no_schedule:
        out["schedule"] = {}
        arr = w.arrivals.numpy()
        policies = [("klpm", oracle.POLICY_KLPM, k) for k in w.ks]
        if name == "streaming":
            policies += [("fcfs", oracle.POLICY_FCFS, 1), ("lpm", oracle.POLICY_LPM, 1)]
        for label, policy, k in policies:
            tree.close()
            tree = build_tree(w)
            t0 = time.time()
            order, unc, ttft, comp = oracle.schedule(qtn, qon, arr, policy, k, 0, 1, w.start_tick,
                                                     oracle.CACHE_TREE, oracle.TIER_UPDATE, tree)
            st = tree.stats()
            key = "%s_k%d" % (label, k)
            out["schedule"][key] = {
                "order_sha256": digest(order.astype("<i4")), "uncached_sha256": digest(unc.astype("<i4")),
                "ttft_sha256": digest(ttft.astype("<i8")), "completion_sha256": digest(comp.astype("<i8")),
                "order_head": order[:16].tolist(), "order_tail": order[-16:].tolist(),
                "total_uncached": int(unc.astype(np.int64).sum()), "ttft_max": int(ttft.max()),
                "ttft_p50": int(np.sort(ttft)[len(ttft) // 2]), "ttft_p99": int(np.sort(ttft)[(len(ttft) * 99) // 100]),
                "tree_after": st}
            print("%s scheduled in %.0f s: %s" % (key, time.time() - t0, out["schedule"][key]["tree_after"]), flush=True)
            with open(path, "w") as f:
                json.dump(out, f, indent=1)
    with open(path, "w") as f:
        json.dump(out, f, indent=1)
    print("wrote", path)


if __name__ == "__main__":
    main()
