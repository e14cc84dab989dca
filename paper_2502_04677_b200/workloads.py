"""Seeded synthetic query streams shaped like the paper's workloads.

This module only *generates inputs*: prompts (int32 token strings in CSR form),
arrival ticks and workload parameters.  It contains none of the scheduler's
arithmetic (no matching, no selection, no cost model) and is the one module the
CPU oracle's tests and the CUDA path both consume, so that both sides see the
very same arrays.

Prompts follow the tree-structured shape of Section 4.1 (a shared base prompt,
a shared user context, a unique tail): every prompt is a concatenation of up to
four *segments*, each segment being a window of a pseudo-random token stream
identified by a 64-bit key.  Two prompts that use the same key for a segment
share those tokens, which is what produces shared prefixes.  Tokens are a pure
function of (key, position), computed with a counter-based integer generator
(the SplitMix64 finaliser), so any slice of any prompt can be materialised on
any device without materialising the rest, and CPU and GPU materialisations
are identical bit for bit.

Arrival times follow Definition 1 (non-negative, one per query); the stream
configurations use a Poisson process (Section 5) quantised to integer ticks.
"""
from __future__ import annotations

import math
from dataclasses import dataclass, field
from typing import List, Optional, Sequence, Tuple

import torch

_M64 = (1 << 64) - 1


def _s64(x: int) -> int:
    """Python int -> the signed 64-bit integer with the same bit pattern."""
    x &= _M64
    return x - (1 << 64) if x >= (1 << 63) else x


_GOLD = _s64(0x9E3779B97F4A7C15)
_MUL1 = _s64(0xBF58476D1CE4E5B9)
_MUL2 = _s64(0x94D049BB133111EB)


def _lsr(z: torch.Tensor, s: int) -> torch.Tensor:
    """Logical shift right of an int64 tensor (torch's >> is arithmetic)."""
    return (z >> s) & ((1 << (64 - s)) - 1)


def mix64(z: torch.Tensor) -> torch.Tensor:
    """SplitMix64 output function on an int64 tensor (wrapping arithmetic)."""
    z = z + _GOLD
    z = (z ^ _lsr(z, 30)) * _MUL1
    z = (z ^ _lsr(z, 27)) * _MUL2
    return z ^ _lsr(z, 31)


def mix64_int(z: int) -> int:
    """The same function on one Python integer (unsigned 64-bit result)."""
    z = (z + 0x9E3779B97F4A7C15) & _M64
    z = ((z ^ (z >> 30)) * 0xBF58476D1CE4E5B9) & _M64
    z = ((z ^ (z >> 27)) * 0x94D049BB133111EB) & _M64
    return z ^ (z >> 31)


def stream_key(seed: int, kind: int, ident: torch.Tensor) -> torch.Tensor:
    """64-bit key of token stream number `ident` of family `kind`."""
    base = _s64(mix64_int((seed * 0x100 + kind) & _M64))
    return mix64(ident.to(torch.int64) * _GOLD + base)


def uniform_u53(seed: int, kind: int, n: int) -> torch.Tensor:
    """n integers uniform in [0, 2^53), one per index, on the CPU."""
    k = stream_key(seed, kind, torch.arange(n, dtype=torch.int64))
    return _lsr(mix64(k), 11)


def uniform_int(seed: int, kind: int, n: int, lo: int, hi: int) -> torch.Tensor:
    """n integers uniform in [lo, hi] (inclusive), on the CPU."""
    return lo + uniform_u53(seed, kind, n) % (hi - lo + 1)


def zipf_index(seed: int, kind: int, n: int, n_items: int, s: float) -> torch.Tensor:
    """n item indices in [0, n_items) with P(rank r) ~ r^-s (integer CDF table)."""
    w = torch.arange(1, n_items + 1, dtype=torch.float64).pow(-s)
    cdf = torch.cumsum(w, 0)
    cdf = (cdf / cdf[-1] * float(1 << 53)).to(torch.int64)
    cdf[-1] = 1 << 53
    u = uniform_u53(seed, kind, n)
    return torch.searchsorted(cdf, u, right=True).clamp_(max=n_items - 1)


def poisson_arrivals(seed: int, kind: int, n: int, rate_per_sec: float, ticks_per_sec: int) -> torch.Tensor:
    """Arrival ticks of a Poisson process: integer-quantised exponential gaps."""
    u = (uniform_u53(seed, kind, n).to(torch.float64) + 0.5) / float(1 << 53)
    gaps = torch.floor(-torch.log(u) * (ticks_per_sec / rate_per_sec)).to(torch.int64)
    return torch.cumsum(gaps, 0)


@dataclass
class SegmentedPrompts:
    """n prompts, each the concatenation of L stream windows.

    seg_key[l][i]  : key of the stream prompt i reads in segment l
    seg_end[l][i]  : position in prompt i where segment l ends (non-decreasing
                     in l; the last one is the prompt length)
    diverge        : if set, the first token of the last segment is forced to
                     differ from the token the previous segment's stream would
                     have produced at that position (a guaranteed mismatch one
                     token past the shared part)
    """
    vocab: int
    seg_key: List[torch.Tensor]
    seg_end: List[torch.Tensor]
    diverge: bool = False

    @property
    def n(self) -> int:
        return int(self.seg_end[-1].numel())

    @property
    def lengths(self) -> torch.Tensor:
        return self.seg_end[-1]

    def offsets(self, lo: int = 0, hi: Optional[int] = None) -> torch.Tensor:
        hi = self.n if hi is None else hi
        off = torch.zeros(hi - lo + 1, dtype=torch.int64)
        torch.cumsum(self.lengths[lo:hi], 0, out=off[1:])
        return off

    def total_tokens(self) -> int:
        return int(self.lengths.sum())

    def select(self, idx: torch.Tensor) -> "SegmentedPrompts":
        idx = idx.to(torch.int64)
        return SegmentedPrompts(self.vocab, [k[idx] for k in self.seg_key],
                                [e[idx] for e in self.seg_end], self.diverge)

    def _tokens_range(self, lo: int, hi: int, device) -> torch.Tensor:
        L = len(self.seg_key)
        lens = self.lengths[lo:hi].to(device)
        n = hi - lo
        total = int(lens.sum())
        if total == 0:
            return torch.empty(0, dtype=torch.int32, device=device)
        off = torch.zeros(n + 1, dtype=torch.int64, device=device)
        torch.cumsum(lens, 0, out=off[1:])
        pi = torch.repeat_interleave(torch.arange(n, dtype=torch.int64, device=device), lens,
                                     output_size=total)
        j = torch.arange(total, dtype=torch.int64, device=device) - off[pi]
        keys = [k[lo:hi].to(device) for k in self.seg_key]
        ends = [e[lo:hi].to(device) for e in self.seg_end]
        key = keys[0][pi]
        start = torch.zeros_like(j)
        for l in range(1, L):
            e = ends[l - 1][pi]
            sel = j >= e
            key = torch.where(sel, keys[l][pi], key)
            start = torch.where(sel, e, start)
        tok = _lsr(mix64(key + (j - start)), 33) % self.vocab
        del key, start, pi, j
        if self.diverge and L >= 2:
            cut = ends[L - 2]
            has = cut < ends[L - 1]
            pidx = torch.nonzero(has).flatten()
            if pidx.numel():
                pstart = ends[L - 3][pidx] if L >= 3 else torch.zeros_like(pidx)
                c = cut[pidx]
                cont = _lsr(mix64(keys[L - 2][pidx] + (c - pstart)), 33) % self.vocab
                at = off[pidx] + c
                cur = tok[at]
                tok[at] = torch.where(cur == cont, (cur + 1) % self.vocab, cur)
        return tok.to(torch.int32)

    def materialize(self, device="cpu", lo: int = 0, hi: Optional[int] = None,
                    chunk_tokens: int = 1 << 25) -> Tuple[torch.Tensor, torch.Tensor]:
        """Tokens (int32, on `device`) and offsets (int64, on the CPU) of prompts [lo, hi)."""
        hi = self.n if hi is None else hi
        off = self.offsets(lo, hi)
        out = torch.empty(int(off[-1]), dtype=torch.int32, device=device)
        self.materialize_into(out, lo, hi, chunk_tokens)
        return out, off

    def materialize_into(self, out: torch.Tensor, lo: int, hi: int, chunk_tokens: int = 1 << 25) -> None:
        off = self.offsets(lo, hi)
        a = lo
        while a < hi:
            # largest b with off[b-lo] - off[a-lo] <= chunk_tokens, at least one prompt
            limit = int(off[a - lo]) + chunk_tokens
            b = int(torch.searchsorted(off, torch.tensor(limit), right=True)) - 1 + lo
            b = max(a + 1, min(b, hi))
            out[int(off[a - lo]):int(off[b - lo])] = self._tokens_range(a, b, out.device)
            a = b


@dataclass
class Workload:
    """One synthetic configuration: the cached prompts, the query stream and its parameters."""
    name: str
    vocab: int
    prefill: SegmentedPrompts           # prompts already in the radix tree when the stream starts
    queries: SegmentedPrompts           # the query stream x_i
    arrivals: torch.Tensor              # t_i, int64 ticks (CPU)
    ticks_per_sec: int
    ks: Sequence[int]                   # k values of k-LPM this configuration is run with
    start_tick: int                     # tick at which processing starts
    budget_tokens: int = 0              # KV-cache budget in tokens, 0 = unbounded
    notes: str = ""
    recipe: dict = field(default_factory=dict)


# stream families (the `kind` argument of stream_key / uniform_*)
_K_PREFIX, _K_SUFFIX_TREE, _K_SUFFIX_Q = 1, 2, 3
_K_LEN_PREFIX, _K_LEN_SUF_TREE, _K_LEN_SUF_Q = 4, 5, 6
_K_PICK_TREE, _K_PICK_Q, _K_ARRIVAL = 7, 8, 9
_K_SYS, _K_BLOCK, _K_DOC, _K_LEN_DOC = 10, 11, 12, 13
_K_UNIQUE_Q, _K_LEN_UNIQUE, _K_IS_UNIQUE = 14, 15, 16
_K_TRUNK, _K_CUT_TREE, _K_CUT_Q = 17, 18, 19


def _two_level(seed, vocab, n, prefix_len, pick, suffix_kind, len_kind, suf_lo, suf_hi, id_base=0):
    """prompt i = prefix[pick[i]] + unique suffix i."""
    n_prefix = prefix_len.numel()
    pkeys = stream_key(seed, _K_PREFIX, torch.arange(n_prefix))
    suf_len = uniform_int(seed, len_kind, n, suf_lo, suf_hi)
    skeys = stream_key(seed, suffix_kind, torch.arange(n) + id_base)
    e0 = prefix_len[pick]
    return SegmentedPrompts(vocab, [pkeys[pick], skeys], [e0, e0 + suf_len])


def tiny(seed: int = 0, n_queries: int = 1000, n_prefill: int = 2000) -> Workload:
    """1,000 waiting queries over 8 shared 512-token prefixes, k = 2."""
    vocab = 32000
    plen = torch.full((8,), 512, dtype=torch.int64)
    tree = _two_level(seed, vocab, n_prefill, plen, uniform_int(seed, _K_PICK_TREE, n_prefill, 0, 7),
                      _K_SUFFIX_TREE, _K_LEN_SUF_TREE, 64, 256)
    q = _two_level(seed, vocab, n_queries, plen, uniform_int(seed, _K_PICK_Q, n_queries, 0, 7),
                   _K_SUFFIX_Q, _K_LEN_SUF_Q, 64, 256)
    tps = 10_000
    arr = poisson_arrivals(seed, _K_ARRIVAL, n_queries, 50.0, tps)
    return Workload("tiny", vocab, tree, q, arr, tps, (2,), int(arr.max()) if n_queries else 0,
                    recipe=dict(seed=seed, prefixes=8, prefix_len=512, suffix="U[64,256]", rate=50))


def medium(seed: int = 1, scale: float = 1.0) -> Workload:
    """32,768 waiting queries over 64 shared prefixes U[1024,4096]; tree of 100,000 prompts."""
    vocab = 128_256
    nq = max(1, int(32_768 * scale))
    npre = max(1, int(100_000 * scale))
    plen = uniform_int(seed, _K_LEN_PREFIX, 64, 1024, 4096)
    tree = _two_level(seed, vocab, npre, plen, uniform_int(seed, _K_PICK_TREE, npre, 0, 63),
                      _K_SUFFIX_TREE, _K_LEN_SUF_TREE, 128, 1024)
    q = _two_level(seed, vocab, nq, plen, uniform_int(seed, _K_PICK_Q, nq, 0, 63),
                   _K_SUFFIX_Q, _K_LEN_SUF_Q, 128, 1024)
    tps = 10_000
    arr = poisson_arrivals(seed, _K_ARRIVAL, nq, 1000.0, tps)
    return Workload("medium", vocab, tree, q, arr, tps, (1, 2, 4, 8), int(arr.max()),
                    recipe=dict(seed=seed, scale=scale, prefixes=64, prefix_len="U[1024,4096]",
                                suffix="U[128,1024]"))


def _hier(seed, vocab, n, leaf, doc_len, q_kind, qlen_kind, id_base):
    """prompt = system[leaf/512] + block[leaf/16] + doc[leaf] + unique question."""
    sysk = stream_key(seed, _K_SYS, torch.arange(4))
    blkk = stream_key(seed, _K_BLOCK, torch.arange(4 * 32))
    dock = stream_key(seed, _K_DOC, torch.arange(4 * 32 * 16))
    qk = stream_key(seed, q_kind, torch.arange(n) + id_base)
    qlen = uniform_int(seed, qlen_kind, n, 32, 128)
    e0 = torch.full((n,), 2048, dtype=torch.int64)
    e1 = e0 + 1024
    e2 = e1 + doc_len[leaf]
    return SegmentedPrompts(vocab, [sysk[leaf // 512], blkk[leaf // 16], dock[leaf], qk],
                            [e0, e1, e2, e2 + qlen])


def hierarchical(seed: int = 2, scale: float = 1.0) -> Workload:
    """Three-level sharing (4 system prompts x 32 few-shot blocks x 16 documents), Zipf(1.1) leaves."""
    vocab = 128_256
    nq = max(1, int(65_536 * scale))
    npre = max(1, int(1_000_000 * scale))
    doc_len = uniform_int(seed, _K_LEN_DOC, 2048, 512, 4096)
    tree = _hier(seed, vocab, npre, zipf_index(seed, _K_PICK_TREE, npre, 2048, 1.1), doc_len,
                 _K_SUFFIX_TREE, _K_LEN_SUF_TREE, 0)
    q = _hier(seed, vocab, nq, zipf_index(seed, _K_PICK_Q, nq, 2048, 1.1), doc_len,
              _K_SUFFIX_Q, _K_LEN_SUF_Q, 0)
    tps = 10_000
    arr = poisson_arrivals(seed, _K_ARRIVAL, nq, 1000.0, tps)
    return Workload("hierarchical", vocab, tree, q, arr, tps, (4,), int(arr.max()),
                    recipe=dict(seed=seed, scale=scale, levels="4x2048 / 32x1024 / 16xU[512,4096]",
                                question="U[32,128]", zipf=1.1))


def streaming(seed: int = 3, scale: float = 1.0) -> Workload:
    """Poisson 200 queries/s for 600 s; 70 % shared-prefix (256 prefixes, Zipf 1.0), 30 % unique."""
    vocab = 128_256
    tps = 330_000
    n = max(1, int(200 * 600 * scale))
    arr = poisson_arrivals(seed, _K_ARRIVAL, n, 200.0, tps)
    plen = uniform_int(seed, _K_LEN_PREFIX, 256, 1024, 4096)
    pick = zipf_index(seed, _K_PICK_Q, n, 256, 1.0)
    unique = uniform_u53(seed, _K_IS_UNIQUE, n) % 10 >= 7
    pkeys = stream_key(seed, _K_PREFIX, torch.arange(256))
    suf_len = torch.where(unique, uniform_int(seed, _K_LEN_UNIQUE, n, 256, 8192),
                          uniform_int(seed, _K_LEN_SUF_Q, n, 128, 1024))
    e0 = torch.where(unique, torch.zeros(n, dtype=torch.int64), plen[pick])
    q = SegmentedPrompts(vocab, [pkeys[pick], stream_key(seed, _K_SUFFIX_Q, torch.arange(n))],
                         [e0, e0 + suf_len])
    empty = SegmentedPrompts(vocab, [torch.zeros(0, dtype=torch.int64)] * 2,
                             [torch.zeros(0, dtype=torch.int64)] * 2)
    return Workload("streaming", vocab, empty, q, arr, tps, (4,), 0,
                    budget_tokens=max(16_384, int(50_000_000 * scale)),
                    recipe=dict(seed=seed, scale=scale, rate=200, seconds=600 * scale, shared="70%",
                                prefixes=256, zipf=1.0, unique="U[256,8192]"))


def adversarial(seed: int = 4, scale: float = 1.0) -> Workload:
    """Near-mismatch prompts on deep edges: trunk[r][:p] + tail, p ~ U[1,16384]."""
    vocab = 128_256
    n_trunk = max(1, int(12_288 * scale))
    npre = max(1, int(2_000_000 * scale))
    nq = max(1, int(262_144 * scale))
    tk = stream_key(seed, _K_TRUNK, torch.arange(n_trunk))

    def make(n, pick_kind, cut_kind, tail_kind, len_kind, diverge):
        r = uniform_int(seed, pick_kind, n, 0, n_trunk - 1)
        cut = uniform_int(seed, cut_kind, n, 1, 16_384)
        tail = uniform_int(seed, len_kind, n, 36, 164)
        return SegmentedPrompts(vocab, [tk[r], stream_key(seed, tail_kind, torch.arange(n))],
                                [cut, cut + tail], diverge)

    tree = make(npre, _K_PICK_TREE, _K_CUT_TREE, _K_SUFFIX_TREE, _K_LEN_SUF_TREE, False)
    q = make(nq, _K_PICK_Q, _K_CUT_Q, _K_SUFFIX_Q, _K_LEN_SUF_Q, True)
    tps = 10_000
    arr = poisson_arrivals(seed, _K_ARRIVAL, nq, 1000.0, tps)
    return Workload("adversarial", vocab, tree, q, arr, tps, (4,), int(arr.max()),
                    recipe=dict(seed=seed, scale=scale, trunks=n_trunk, trunk_len=16_384,
                                cut="U[1,16384]", tail="U[36,164]"))


def prefix_ratio(u: int, d: int, seed: int = 5, n: int = 2000, rep: int = 4, scale: float = 1.0) -> Workload:
    """The prefix-to-prompt ratio experiment of Appendix C.2 under the cost model: a regular-arrival-style
    queue (Definition 3) of n random-string prompts (user)(doc), each user substring of length u shared by
    `rep` prompts, each doc substring of length d unique, shuffled, arriving as a Poisson stream of 80
    queries per second; empty cache; policies k = 1, 4 and LPM.  One tick = one prefilled token at a rate
    of 300,000 tokens per second (offered load about 1 for u = d = 3000 with perfect reuse)."""
    vocab = 128_256
    n = max(rep, int(n * scale) // rep * rep)
    tps = 300_000
    user = torch.arange(n) // rep
    order = torch.argsort(uniform_u53(seed, _K_PICK_Q, n))          # random shuffle of the queue
    user = user[order]
    ukeys = stream_key(seed, _K_PREFIX, torch.arange(n // rep))
    dkeys = stream_key(seed, _K_SUFFIX_Q, torch.arange(n))
    e0 = torch.full((n,), u, dtype=torch.int64)
    q = SegmentedPrompts(vocab, [ukeys[user], dkeys], [e0, e0 + d])
    empty = SegmentedPrompts(vocab, [torch.zeros(0, dtype=torch.int64)] * 2, [torch.zeros(0, dtype=torch.int64)] * 2)
    arr = poisson_arrivals(seed, _K_ARRIVAL, n, 80.0, tps)
    return Workload("ratio_%d_%d" % (u, d), vocab, empty, q, arr, tps, (4,), 0,
                    recipe=dict(seed=seed, scale=scale, u=u, d=d, n=n, rep=rep, rate=80))


def _ratio(u, d):
    def make(seed: int = 5, scale: float = 1.0) -> Workload:
        return prefix_ratio(u, d, seed=seed, scale=scale)
    return make


WORKLOADS = {"tiny": tiny, "medium": medium, "hierarchical": hierarchical,
             "streaming": streaming, "adversarial": adversarial,
             "ratio_1000_5000": _ratio(1000, 5000), "ratio_3000_3000": _ratio(3000, 3000),
             "ratio_5000_1000": _ratio(5000, 1000)}


# ---------------------------------------------------------------------------
# Small explicit queues used to pin the oracle (plain Python lists of ints).
# ---------------------------------------------------------------------------

def regular_arrival_shuffled_queue(n: int, rep: int, u: int, d: int, s: int,
                                   sigma: Sequence[int]) -> Tuple[List[List[int]], List[int]]:
    """Definition 3: n prompts (user)(doc); each user substring (length u) is shared by `rep`
    prompts, each doc substring (length d) is unique; all substrings start with distinct tokens.
    sigma is a permutation of 1..n; prompt i arrives at tick s * sigma[i]."""
    assert n % rep == 0 and sorted(sigma) == list(range(1, n + 1))
    n_user = n // rep
    prompts = []
    for i in range(n):
        usr = i % n_user          # x_1=(u1,d1), x_2=(u2,d2), x_3=(u1,d3), ... as in the toy example
        user = [1 + usr] + [0] * (u - 1) if u > 0 else []
        doc = [1 + n_user + i] + [0] * (d - 1) if d > 0 else []
        prompts.append(user + doc)
    return prompts, [s * sigma[i] for i in range(n)]


def three_partition_gadget(a: Sequence[int], m: int, H: int) -> Tuple[List[List[int]], List[int], int, List[str]]:
    """Query stream of the NP-hardness construction (Theorem 1) for a 3-PARTITION instance.
    Returns prompts, arrival ticks, the TTFT constraint T = (m + m^2) H and a label per query."""
    assert len(a) == 3 * m and sum(a) == m * H
    T = (m + m * m) * H
    prompts, arrivals, labels = [], [], []
    ch = 1
    for ai in a:                                   # X: unique character, length a_i, arrive at T
        prompts.append([ch] * ai); arrivals.append(T); labels.append("x"); ch += 1
    ych = []
    for i in range(1, m + 1):                      # Y: length mH, arrive at i(H + mH)
        prompts.append([ch] * (m * H)); arrivals.append(i * (H + m * H)); labels.append(f"y{i}")
        ych.append(ch); ch += 1
    for i in range(1, m + 1):                      # Z: same content as y_i, arrive at T + i(H + mH)
        prompts.append([ych[i - 1]] * (m * H)); arrivals.append(T + i * (H + m * H)); labels.append(f"z{i}")
    prompts.append([ch] * T); arrivals.append(0); labels.append("w1"); ch += 1
    prompts.append([ch] * T); arrivals.append(2 * T); labels.append("w2")
    return prompts, arrivals, T, labels


def to_csr(prompts: Sequence[Sequence[int]]) -> Tuple[torch.Tensor, torch.Tensor]:
    """List of token lists -> (tokens int32, offsets int64)."""
    off = [0]
    flat: List[int] = []
    for p in prompts:
        flat.extend(p)
        off.append(len(flat))
    return torch.tensor(flat, dtype=torch.int32), torch.tensor(off, dtype=torch.int64)


def random_small_queue(seed: int, n: int, vocab: int, max_len: int, min_len: int = 0,
                       max_gap: int = 3) -> Tuple[List[List[int]], List[int]]:
    """Random prompts over a tiny alphabet (so that overlaps are frequent) with random arrival gaps."""
    lens = uniform_int(seed, 101, n, min_len, max_len).tolist()
    gaps = uniform_int(seed, 102, n, 0, max_gap).tolist()
    prompts, arrivals, t = [], [], 0
    for i in range(n):
        toks = (uniform_u53(seed * 7919 + i, 103, lens[i]) % vocab).tolist() if lens[i] else []
        prompts.append([int(x) for x in toks])
        t += gaps[i]
        arrivals.append(t)
    return prompts, arrivals
