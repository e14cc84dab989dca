// Device-resident k-LPM scheduling path for sm_100a: flattened radix tree, batched longest-prefix
// match, k-LPM selection, schedule replay with LRU eviction.  See include/klpm.h for the ABI.
//
// Layout in HBM
//   nodes   : structure of arrays indexed by node id (0 = root): parent, depth_start, span_len, nchild
//             (int32), span_off, last_access (int64), dead (uint8).  Ids are never reused.
//   pool    : append-only int32 token pool; node v's edge label is pool[span_off[v] .. +span_len[v]).
//             Edges are placed so that span_off = depth_start (mod 4): the pool tokens that pair with
//             query positions 4i..4i+3 are one aligned 128-bit load.  A split never moves tokens, so
//             "pool index of the last matched token" identifies a position in the tree for as long as
//             the tree lives, and the pieces of a leaf that was cut stay one contiguous run
//             (chain_end in the child table, end_node[] per pool token: see walk_chain).
//   children: one open-addressing hash table for the whole tree keyed by (parent id, first token of the
//             child's edge).  An entry is one 32-byte sector and carries what a walk needs for the hop
//             (child id, edge length, edge offset, end of its contiguous run), so a hop costs one
//             dependent sector read.
//   LRU     : last_access holds logical clocks.  Only the node where a processed prompt's cached part
//             ends and its new leaf are stamped; when a leaf is evicted its stamp is handed to its
//             parent if newer.  For every leaf this equals the clock of the last processed prompt
//             whose path covers it, which is all eviction looks at.  clock_owner[c] names the node
//             holding stamp c, so the least recently used leaf is found by a cursor that only moves
//             forward over clock values.
#include <cuda_runtime.h>
#include <stdint.h>
#include <stdio.h>
#include <stdlib.h>
#include <string.h>
#include <atomic>
#include <new>

#include "klpm.h"

#define FULL_MASK 0xffffffffu
#define KLPM_ABI_VERSION 3

namespace {

struct alignas(32) Entry {
    unsigned long long key;   // ((parent + 1) << 32) | first token ; 0 = empty slot
    int32_t child;            // node id, or -1 if the child was evicted (slot is reused on re-insert)
    int32_t span_len;
    int64_t span_off;
    int64_t chain_end;        // pool index one past the contiguous pool run this edge is part of (see walk_chain)
};

struct TreeState {
    long long n_nodes;      // next free node id
    long long pool_used;
    long long tokens_live;
    long long live_nodes;   // root excluded
    long long clock;
    long long lru_cursor;
    long long evictions;
    int status;
    int detail;             // which check recorded the status (a debugging aid, see rt_status_detail)
};

struct TreeDev {
    int32_t* parent;
    int32_t* depth_start;
    int32_t* span_len;
    int32_t* nchild;
    int32_t* first_tok;       // first token of the node's edge (= pool[span_off])
    int64_t* span_off;
    int64_t* last_access;
    uint8_t* dead;
    int32_t* clock_owner;
    Entry* table;
    unsigned long long table_mask;
    int32_t* pool;
    int32_t* end_node;        // per pool index: id of the node whose edge ends with that token, else -1
    TreeState* st;
    long long max_nodes, max_pool, max_clock, budget;
};

// ------------------------------------------------------------------------------------------------
// loads: RO = the kernel never writes what it reads (read-only path), otherwise L2-coherent loads
// ------------------------------------------------------------------------------------------------
template <bool RO> __device__ __forceinline__ int32_t ld32(const int32_t* p) { return RO ? __ldg(p) : __ldcg(p); }
template <bool RO> __device__ __forceinline__ Entry ld_entry(const Entry* e) {
    const int4* p = reinterpret_cast<const int4*>(e);
    int4 a = RO ? __ldg(p) : __ldcg(p);
    int4 b = RO ? __ldg(p + 1) : __ldcg(p + 1);
    Entry r;
    r.key = ((unsigned long long)(unsigned)a.y << 32) | (unsigned)a.x;
    r.child = a.z;
    r.span_len = a.w;
    r.span_off = (int64_t)(((unsigned long long)(unsigned)b.y << 32) | (unsigned)b.x);
    r.chain_end = (int64_t)(((unsigned long long)(unsigned)b.w << 32) | (unsigned)b.z);
    return r;
}

__device__ __forceinline__ unsigned long long make_key(int32_t parent, int32_t tok) {
    return ((unsigned long long)(unsigned)(parent + 1) << 32) | (unsigned)tok;
}
// Table hash: the two key halves are combined with the golden-ratio multiplier and run through the
// 32-bit finaliser of MurmurHash3 (public domain, A. Appleby).  32-bit arithmetic keeps a hop cheap.
__device__ __forceinline__ unsigned long long hash_key(unsigned long long k) {
    unsigned h = (unsigned)(k >> 32) * 0x9E3779B1u + (unsigned)k;
    h ^= h >> 16; h *= 0x85ebca6bu; h ^= h >> 13; h *= 0xc2b2ae35u; h ^= h >> 16;
    return (unsigned long long)h;
}

__device__ __forceinline__ void set_status(TreeState* st, int code, int detail = 0) {
    if (atomicCAS(&st->status, 0, code) == 0) st->detail = detail;
}

// A child lookup that probed every slot of the table without meeting the key or an empty slot gives up; the
// walk then reports a shorter match, and the status word says that it is not to be trusted.
__device__ __noinline__ void probe_limit(const TreeDev& T) {
    if ((threadIdx.x & 31) == 0) set_status(T.st, RT_ERR_LIMIT, 106);
}

// First index in [0, n) where a and b differ, or n.  Warp-cooperative: every lane gets the result.
// Lane l reads elements l, l+32, l+64, ... of each chunk: each load instruction of the warp is one
// contiguous 128-byte request, whatever the 4-byte phase of the two streams.  U * 128 tokens of both
// streams are requested before the first of them is examined, so a long common prefix costs one memory
// latency per U * 128 tokens.
template <bool RO, int U = 4>
__device__ __forceinline__ int32_t first_mismatch(const int32_t* __restrict__ a, const int32_t* __restrict__ b, int32_t n) {
    const int lane = threadIdx.x & 31;
    constexpr int R = 4 * U;
    for (int32_t base = 0; base < n; base += 32 * R) {
        int32_t x[R], y[R];
#pragma unroll
        for (int j = 0; j < R; ++j) {
            int32_t idx = base + j * 32 + lane;
            bool in = idx < n;
            x[j] = in ? ld32<RO>(a + idx) : 0;
            y[j] = in ? ld32<RO>(b + idx) : 0;
        }
#pragma unroll
        for (int j = 0; j < R; ++j) {
            if (base + j * 32 >= n) break;                  // warp-uniform
            unsigned bad = __ballot_sync(FULL_MASK, x[j] != y[j]);
            if (bad) return base + j * 32 + (__ffs(bad) - 1);
        }
    }
    return n;
}

struct Term {
    int32_t m;      // matched tokens
    int32_t node;   // node whose edge holds the last matched token (0 = root)
    int32_t off;    // tokens of that edge matched
    int64_t pos;    // pool index of the last matched token, -1 at the root
    int32_t full;   // 1 if the match ends exactly at the end of that node's edge (or at the root)
};

// Longest prefix of q on a root path.  Warp-cooperative and warp-uniform.  (cur0, m0): a node boundary the walk may
// start from instead of the root -- the first m0 tokens of q are known to end exactly at the end of cur0's edge.
template <bool RO>
__device__ Term walk(const TreeDev& T, const int32_t* __restrict__ q, int32_t len, int32_t cur0 = 0, int32_t m0 = 0) {
    Term t; t.m = m0; t.node = cur0; t.off = 0; t.pos = -1; t.full = 1;
    if (len <= m0) return t;
    unsigned long long key = make_key(cur0, ld32<RO>(q + m0));
    unsigned long long slot = hash_key(key) & T.table_mask;
    Entry c = ld_entry<RO>(T.table + slot);
    for (;;) {
        unsigned long long probes = 0;
        while (c.key != key) {
            if (c.key == 0ULL) return t;
            if (++probes > T.table_mask) { probe_limit(T); return t; }      // no empty slot: cannot happen below load 1
            slot = (slot + 1) & T.table_mask;
            c = ld_entry<RO>(T.table + slot);
        }
        if (c.child < 0) return t;
        const int32_t rem = len - t.m;
        const int32_t n = c.span_len < rem ? c.span_len : rem;
        const bool has_next = c.span_len < rem;
        // issue the probe of the next hop before comparing this edge: it depends only on this entry
        unsigned long long key2 = 0, slot2 = 0;
        Entry nx; nx.key = 0; nx.child = -1; nx.span_len = 0; nx.span_off = 0; nx.chain_end = 0;
        if (has_next) {
            key2 = make_key(c.child, ld32<RO>(q + t.m + c.span_len));
            slot2 = hash_key(key2) & T.table_mask;
            nx = ld_entry<RO>(T.table + slot2);
        }
        const int32_t i = first_mismatch<RO>(q + t.m, T.pool + c.span_off, n);
        t.m += i;
        t.node = c.child;
        t.off = i;
        t.pos = c.span_off + i - 1;     // i >= 1: the first token is the key
        t.full = i == c.span_len;
        if (i < c.span_len || !has_next) return t;
        key = key2; slot = slot2; c = nx;
    }
}

// The walk of the read-only batched kernel on a tree that never evicts (no budget).
//
// A leaf's edge is written to the pool as one contiguous run, and later cuts only put node boundaries
// inside that run: the pieces stay adjacent, each the one child of the previous for the token that
// follows.  So a query that enters such a run at the start of a node matches exactly as far as it agrees
// with the contiguous pool tokens, whatever the number of boundaries it crosses; no child lookup is needed
// inside the run.  Every table entry carries chain_end, the pool index where its run ends, and
// end_node[] tells whether a pool token is the last one of a node: a lookup is only made where the
// comparison stops on a node boundary (another child may continue there) or the run is exhausted.
// The comparison itself is a stream: 128-bit loads of both sides, two 128-token chunks in flight.
//
// Coordinates are depths (token positions in the query).  Every edge is placed so that
// span_off = depth_start (mod 4), hence the pool tokens of depths 4i..4i+3 are one aligned 128-bit load.
// The query side is read with aligned 128-bit loads too and shifted across lanes when the query does not
// start on a 16-byte boundary.  The 16-byte units that hold the query's first and last token are read
// whole: the token buffer must be 16-byte aligned (as cudaMalloc'd memory is).
struct QWin {
    const int32_t* qa;   // q rounded down to 16 bytes
    int32_t s;           // tokens q is past that boundary (0..3)
    int32_t len;
};

// Query tokens are read once and never again: they are loaded with the streaming hint, so that the pool tokens --
// which other queries of the same trunk are about to read -- are what stays in L2.
__device__ __forceinline__ int4 ld_query4(const int4* p) { return __ldcs(p); }

// tokens of depths cb + 4 lane .. + 3 (cb a multiple of 4); zeros where nothing needs to be read
__device__ __forceinline__ int4 qwin_load(const QWin& Q, int32_t cb, int lane) {
    const int4 z = make_int4(0, 0, 0, 0);
    const int32_t p0 = cb + 4 * lane;
    int4 v = (p0 - Q.s < Q.len) ? ld_query4(reinterpret_cast<const int4*>(Q.qa + p0)) : z;
    if (Q.s == 0) return v;                                            // warp-uniform
    int4 e = (cb + 128 - Q.s < Q.len) ? ld_query4(reinterpret_cast<const int4*>(Q.qa + cb + 128)) : z;
    int4 n;
    n.x = __shfl_down_sync(FULL_MASK, v.x, 1); n.y = __shfl_down_sync(FULL_MASK, v.y, 1); n.z = __shfl_down_sync(FULL_MASK, v.z, 1);
    if (lane == 31) { n.x = e.x; n.y = e.y; n.z = e.z; }
    if (Q.s == 1) return make_int4(v.y, v.z, v.w, n.x);
    if (Q.s == 2) return make_int4(v.z, v.w, n.x, n.y);
    return make_int4(v.w, n.x, n.y, n.z);
}

// First depth >= lo of this 128-token chunk (lane l: depths p0 .. p0+3) where A and P differ, or -1.
__device__ __forceinline__ int32_t chunk_mismatch(const int4& A, const int4& P, int32_t p0, int32_t lo) {
    int32_t dx = P.x ^ A.x, dy = P.y ^ A.y, dz = P.z ^ A.z, dw = P.w ^ A.w;
    const int32_t hm = lo - p0;                     // leading tokens of this lane that are before lo
    if (hm > 0) dx = 0;
    if (hm > 1) dy = 0;
    if (hm > 2) dz = 0;
    const int32_t fc = dx ? 0 : dy ? 1 : dz ? 2 : dw ? 3 : 4;
    const unsigned bad = __ballot_sync(FULL_MASK, fc < 4);
    if (!bad) return -1;
    const int L = __ffs(bad) - 1;
    return __shfl_sync(FULL_MASK, p0 + fc, L);
}

// First depth in [lo, hi) where the query differs from pool_d[depth], or hi.  pool_d is the pool pointer
// shifted so that pool_d[p] pairs with depth p; it is 16-byte aligned.
#ifndef KLPM_PREFETCH_DIST
#define KLPM_PREFETCH_DIST 2
#endif
// One 128-token chunk with every bound checked: depths below lo and at or above hi take no part.  Returns the first
// depth where the two sides differ (hi at most), or -1.
__device__ __forceinline__ int32_t compare_chunk_edge(const QWin& Q, const int4* __restrict__ pool4, int32_t cb, int32_t lo, int32_t hi, int lane) {
    const int32_t p = cb + 4 * lane;
    const int4 A = qwin_load(Q, cb, lane);
    int4 P = A;
    if (p + 4 > lo && p < hi) P = __ldg(pool4 + (p >> 2));
    const int32_t r = chunk_mismatch(A, P, p, lo);
    if (r < 0) return -1;
    return r < hi ? r : hi;
}

// Both streams of the chunk KLPM_PREFETCH_DIST ahead are asked into L2 (no register waits for them), so that its
// loads find them there: a warp keeps more than one chunk of memory latency in flight.
__device__ __forceinline__ void prefetch_chunk(const QWin& Q, const int4* __restrict__ pool4, int32_t cb, int32_t hi, int lane) {
#if KLPM_PREFETCH_DIST > 0
    const int32_t pf = cb + 128 * KLPM_PREFETCH_DIST + 4 * lane;
    if (pf < hi) {
        asm volatile("prefetch.global.L2 [%0];" ::"l"(pool4 + (pf >> 2)));
        asm volatile("prefetch.global.L2 [%0];" ::"l"(Q.qa + pf));
    }
#endif
}

__device__ __forceinline__ int32_t compare_run(const QWin& Q, const int32_t* __restrict__ pool_d, int32_t lo, int32_t hi, int lane) {
    const int4* __restrict__ pool4 = reinterpret_cast<const int4*>(pool_d);
    const int4* __restrict__ qa4 = reinterpret_cast<const int4*>(Q.qa);
    int32_t cb = lo & ~127;
    // the chunk that holds lo
    prefetch_chunk(Q, pool4, cb, hi, lane);
    int32_t r = compare_chunk_edge(Q, pool4, cb, lo, hi, lane);
    if (r >= 0) return r;
    cb += 128;
    // chunks that lie wholly inside [lo, hi): nothing to mask, nothing to bound, and the exact position of a difference
    // is only worked out once a difference has been seen
    for (; cb + 128 <= hi; cb += 128) {
        prefetch_chunk(Q, pool4, cb, hi, lane);
        const int32_t i4 = (cb >> 2) + lane;
        int4 v = ld_query4(qa4 + i4);
        const int4 P = __ldg(pool4 + i4);
        if (Q.s != 0) {                                                    // warp-uniform
            const int4 e = ld_query4(qa4 + (cb >> 2) + 32);
            int32_t nx = __shfl_down_sync(FULL_MASK, v.x, 1), ny = __shfl_down_sync(FULL_MASK, v.y, 1), nz = __shfl_down_sync(FULL_MASK, v.z, 1);
            if (lane == 31) { nx = e.x; ny = e.y; nz = e.z; }
            if (Q.s == 1) v = make_int4(v.y, v.z, v.w, nx);
            else if (Q.s == 2) v = make_int4(v.z, v.w, nx, ny);
            else v = make_int4(v.w, nx, ny, nz);
        }
        const int32_t dx = v.x ^ P.x, dy = v.y ^ P.y, dz = v.z ^ P.z, dw = v.w ^ P.w;
        const unsigned bad = __ballot_sync(FULL_MASK, (dx | dy | dz | dw) != 0);
        if (bad) {
            const int32_t fc = dx ? 0 : dy ? 1 : dz ? 2 : 3;
            return __shfl_sync(FULL_MASK, cb + 4 * lane + fc, __ffs(bad) - 1);
        }
    }
    // the ragged end
    if (cb < hi) {
        r = compare_chunk_edge(Q, pool4, cb, lo, hi, lane);
        if (r >= 0) return r;
    }
    return hi;
}

// id of the live node whose edge ends with pool token `pos`, or -1.  Entries of end_node[] can be stale
// after a rollback, so a candidate is checked against the node arrays.
struct EndIndex {             // what is needed to resolve end_node[] entries, passed by value
    const int32_t* end_node; const int64_t* span_off; const int32_t* span_len; const uint8_t* dead;
    const TreeState* st;
};
__device__ __forceinline__ EndIndex end_index(const TreeDev& T) {
    EndIndex X; X.end_node = T.end_node; X.span_off = T.span_off; X.span_len = T.span_len; X.dead = T.dead; X.st = T.st;
    return X;
}
__device__ __forceinline__ int32_t node_ending_at(const EndIndex X, int64_t pos, long long n_nodes) {
    const int32_t e = __ldg(X.end_node + pos);
    if (e <= 0 || e >= n_nodes) return -1;
    if (__ldg(X.span_off + e) + __ldg(X.span_len + e) - 1 != pos || __ldg(X.dead + e)) return -1;
    return e;
}

// The node of this run whose edge ends first after pool token `pos` (the match stopped inside its edge).
__device__ __noinline__ int32_t node_after(const EndIndex X, int64_t pos, int64_t chain_end) {
    const int lane = threadIdx.x & 31;
    const long long n_nodes = *reinterpret_cast<const volatile long long*>(&X.st->n_nodes);
    for (int64_t p = pos + 1; p < chain_end; p += 32) {
        const int32_t cand = (p + lane < chain_end) ? node_ending_at(X, p + lane, n_nodes) : -1;
        const unsigned hit = __ballot_sync(FULL_MASK, cand >= 0);
        if (hit) return __shfl_sync(FULL_MASK, cand, __ffs(hit) - 1);
    }
    return -1;
}

// Returns the match length; *node / *off (where the match ended) are filled when want_node is set.
// With WANT_POS, *last_pos receives the pool index of the last matched token (-1 if nothing matched) and
// *last_end the end of the contiguous run that token lies in (what node_after needs to name the node later).
template <bool WANT_POS = false>
__device__ __forceinline__ int32_t walk_chain(const TreeDev& T, const int32_t* __restrict__ q, int32_t len, bool want_node,
                              int32_t* node, int32_t* off, int64_t* last_pos = nullptr, int64_t* last_end = nullptr) {
    const int lane = threadIdx.x & 31;
    *node = 0; *off = 0;
    if (WANT_POS) { *last_pos = -1; *last_end = 0; }
    if (len <= 0) return 0;
    QWin Q;
    Q.s = (int32_t)((reinterpret_cast<uintptr_t>(q) >> 2) & 3);
    Q.qa = q - Q.s;
    Q.len = len;
    int32_t m = 0, cur = 0;
    for (;;) {
        const unsigned long long key = make_key(cur, __ldg(q + m));
        unsigned long long slot = hash_key(key) & T.table_mask;
        Entry c = ld_entry<true>(T.table + slot);
        unsigned long long probes = 0;
        while (c.key != key) {
            if (c.key == 0ULL) return m;
            if (++probes > T.table_mask) { probe_limit(T); return m; }      // no empty slot: cannot happen below load 1
            slot = (slot + 1) & T.table_mask;
            c = ld_entry<true>(T.table + slot);
        }
        if (c.child < 0) return m;
        int64_t run = c.chain_end - c.span_off;
        if (run > (int64_t)(len - m)) run = len - m;
        const int32_t x = compare_run(Q, T.pool + (c.span_off - (int64_t)m), m, m + (int32_t)run, lane);
        const int64_t pos = c.span_off + (x - m) - 1;          // x > m: the first token is the key
        m = x;
        if (WANT_POS) { *last_pos = pos; *last_end = c.chain_end; }
        const int32_t e = node_ending_at(end_index(T), pos, *reinterpret_cast<const volatile long long*>(&T.st->n_nodes));
        if (e < 0) {                                           // stopped inside an edge
            if (want_node) {
                const int32_t f = node_after(end_index(T), pos, c.chain_end);
                if (f >= 0) { *node = f; *off = m - __ldg(T.depth_start + f); }
            }
            return m;
        }
        if (want_node) { *node = e; *off = __ldg(T.span_len + e); }
        if (m >= len) return m;
        cur = e;
    }
}

// ------------------------------------------------------------------------------------------------
// single-thread tree updates (callers serialise them)
// ------------------------------------------------------------------------------------------------
__device__ long long table_find(const TreeDev& T, int32_t parent, int32_t tok) {
    unsigned long long key = make_key(parent, tok);
    unsigned long long slot = hash_key(key) & T.table_mask;
    for (unsigned long long probes = 0; probes <= T.table_mask; ++probes) {
        unsigned long long k = __ldcg(&T.table[slot].key);
        if (k == key) return (long long)slot;
        if (k == 0ULL) return -1;
        slot = (slot + 1) & T.table_mask;
    }
    return -1;
}

__device__ bool table_put(const TreeDev& T, int32_t parent, int32_t tok, int32_t child, int32_t span_len, int64_t span_off,
                          int64_t chain_end) {
    unsigned long long key = make_key(parent, tok);
    unsigned long long slot = hash_key(key) & T.table_mask;
    for (unsigned long long probes = 0; probes <= T.table_mask; ++probes) {
        unsigned long long k = __ldcg(&T.table[slot].key);
        if (k == key || k == 0ULL) {
            Entry* e = T.table + slot;
            e->child = child; e->span_len = span_len; e->span_off = span_off; e->chain_end = chain_end;
            e->key = key;
            return true;
        }
        slot = (slot + 1) & T.table_mask;
    }
    return false;
}

// What a caller has already read for an insertion, so that the serial part need not wait for memory again:
// the tokens that key the table operations and the keys seen in the slots those operations probe first.
struct InsertPre {
    int32_t xm, pt, ft;                       // x[m]; pool token just below the cut; first token of the cut edge
    unsigned long long k_leaf, k_low, k_par;  // keys seen in the first slots of (end, xm), (upper, pt), (parent, ft)
};

__device__ long long table_find_seen(const TreeDev& T, int32_t parent, int32_t tok, unsigned long long seen) {
    const unsigned long long key = make_key(parent, tok);
    if (seen == key) return (long long)(hash_key(key) & T.table_mask);
    return table_find(T, parent, tok);
}

// table_put that trusts `seen` for the first slot unless that slot is `taken` (written since it was read).
__device__ long long table_put_seen(const TreeDev& T, int32_t parent, int32_t tok, int32_t child, int32_t span_len, int64_t span_off,
                                   int64_t chain_end, unsigned long long seen, long long taken) {
    const unsigned long long key = make_key(parent, tok);
    unsigned long long slot = hash_key(key) & T.table_mask;
    bool first = (long long)slot != taken;
    for (unsigned long long probes = 0; probes <= T.table_mask; ++probes) {
        const unsigned long long k = first ? seen : __ldcg(&T.table[slot].key);
        first = false;
        if (k == key || k == 0ULL) {
            Entry* e = T.table + slot;
            e->child = child; e->span_len = span_len; e->span_off = span_off; e->chain_end = chain_end;
            e->key = key;
            return (long long)slot;
        }
        slot = (slot + 1) & T.table_mask;
    }
    return -1;
}

// Node boundary `o` tokens into v's edge (0 < o < span_len[v]): a new node takes the upper part and v's
// place under v's parent; v keeps the lower part, its children and its id.  Returns the new node;
// *low_slot receives the table slot that now holds (new node, first token of the lower part).
__device__ int32_t split_node(const TreeDev& T, int32_t v, int32_t o, const InsertPre* pre, long long* low_slot) {
    TreeState* S = T.st;
    int32_t u = (int32_t)S->n_nodes++;
    S->live_nodes++;
    int32_t par = T.parent[v], ds = T.depth_start[v], len = T.span_len[v];
    int64_t off = T.span_off[v];
    T.parent[u] = par; T.depth_start[u] = ds; T.span_off[u] = off; T.span_len[u] = o;
    T.nchild[u] = 1; T.dead[u] = 0; T.last_access[u] = T.last_access[v];
    const int32_t ft = pre ? pre->ft : __ldcg(T.pool + off);
    const int32_t pt = pre ? pre->pt : __ldcg(T.pool + off + o);
    T.first_tok[u] = ft; T.first_tok[v] = pt;
    const long long slot = pre ? table_find_seen(T, par, ft, pre->k_par) : table_find(T, par, ft);
    int64_t chain_end = off + len;
    if (slot >= 0) { T.table[slot].child = u; T.table[slot].span_len = o; chain_end = T.table[slot].chain_end; }
    else set_status(S, RT_ERR_LIMIT, 101);
    T.span_off[v] = off + o; T.span_len[v] = len - o; T.depth_start[v] = ds + o; T.parent[v] = u;
    const long long ls = pre ? table_put_seen(T, u, pt, v, len - o, off + o, chain_end, pre->k_low, -1)
                             : table_put_seen(T, u, pt, v, len - o, off + o, chain_end, 0ULL, (long long)(hash_key(make_key(u, pt)) & T.table_mask));
    if (ls < 0) set_status(S, RT_ERR_CAPACITY);
    *low_slot = ls;
    T.end_node[off + o - 1] = u;
    return u;
}

__device__ void evict_leaf(const TreeDev& T, int32_t v) {
    TreeState* S = T.st;
    int32_t P = T.parent[v];
    T.dead[v] = 1;
    long long slot = table_find(T, P, __ldcg(T.pool + T.span_off[v]));
    if (slot >= 0) T.table[slot].child = -1;
    T.nchild[P]--;
    S->tokens_live -= T.span_len[v];
    S->live_nodes--;
    S->evictions++;
    if (P != 0 && T.last_access[v] >= T.last_access[P]) {
        T.last_access[P] = T.last_access[v];
        T.clock_owner[T.last_access[v]] = P;
    }
}

struct InsertOut {
    int32_t leaf;      // id of the new leaf, -1 if the prompt was fully cached
    int32_t unc;       // tokens to copy into the pool
    int64_t leaf_off;  // pool offset of the new leaf's edge
    int32_t evicted;   // 1 if any leaf was evicted
    int32_t ok;        // 0 if the prompt could not be stored (status word says why)
};

// Store prompt x (|x| = len) whose cached part is m tokens long and ends in `hint` or an ancestor of it.
// Everything except copying the new leaf's tokens into the pool.  One thread.
__device__ void insert_serial(const TreeDev& T, const int32_t* x, int32_t len, int32_t m, int32_t hint, InsertOut* out,
                              const InsertPre* pre = nullptr) {
    TreeState* S = T.st;
    out->leaf = -1; out->unc = 0; out->leaf_off = 0; out->evicted = 0; out->ok = 0;
    if (S->clock + 1 >= T.max_clock || S->n_nodes + 2 > T.max_nodes) { set_status(S, RT_ERR_CAPACITY); return; }
    const long long clock = ++S->clock;
    int32_t a = hint;
    while (a != 0 && m <= T.depth_start[a]) a = T.parent[a];
    const int32_t o = a == 0 ? 0 : m - T.depth_start[a];
    int32_t end = a;
    long long low_slot = -1;
    if (a != 0 && o < T.span_len[a]) end = split_node(T, a, o, pre, &low_slot);
    if (end != 0) { T.last_access[end] = clock; T.clock_owner[clock] = end; }
    const int32_t unc = len - m;
    if (T.budget > 0) {
        while (S->tokens_live + unc > T.budget) {
            long long cur = S->lru_cursor;
            int32_t victim = -1;
            while (cur < clock) {
                int32_t v = T.clock_owner[cur];
                if (v > 0 && !T.dead[v] && T.last_access[v] == cur && T.nchild[v] == 0) { victim = v; break; }
                ++cur;
            }
            S->lru_cursor = cur;
            if (victim < 0) { set_status(S, RT_ERR_BUDGET); return; }
            evict_leaf(T, victim);
            out->evicted = 1;
        }
    }
    if (unc > 0) {
        if (S->pool_used + unc + 6 > T.max_pool) { set_status(S, RT_ERR_CAPACITY); return; }
        int32_t leaf = (int32_t)S->n_nodes++;
        const int64_t off = ((S->pool_used + 3) & ~3LL) + (m & 3);    // span_off = depth_start (mod 4)
        S->pool_used = off + unc;
        T.parent[leaf] = end; T.depth_start[leaf] = m; T.span_off[leaf] = off; T.span_len[leaf] = unc;
        T.nchild[leaf] = 0; T.dead[leaf] = 0; T.last_access[leaf] = clock;
        T.clock_owner[clock] = leaf;
        T.nchild[end]++;
        const int32_t xm = pre ? pre->xm : __ldcg(x + m);
        T.first_tok[leaf] = xm;
        const long long put = pre ? table_put_seen(T, end, xm, leaf, unc, off, off + unc, pre->k_leaf, low_slot)
                                  : (table_put(T, end, xm, leaf, unc, off, off + unc) ? 0 : -1);
        if (put < 0) { set_status(S, RT_ERR_CAPACITY); return; }
        T.end_node[off + unc - 1] = leaf;
        S->tokens_live += unc;
        S->live_nodes++;
        out->leaf = leaf; out->unc = unc; out->leaf_off = off;
    }
    out->ok = 1;
}

// ------------------------------------------------------------------------------------------------
// rt_match_batch
// ------------------------------------------------------------------------------------------------
#ifndef KLPM_MATCH_MIN_BLOCKS
#define KLPM_MATCH_MIN_BLOCKS 8
#endif
// One warp per query, queries handed out by an atomic counter (persistent grid).
// Trees without a budget: stream along contiguous pool runs.
//
// Queries are taken in the order of `perm` when it is given: the host buckets them by their first token first, so
// that queries which start down the same root child -- and therefore read the same pool tokens -- are in flight
// at the same time and all but the first of them find those tokens in L2.
//
// With STATE the kernel also records, per query, what the scheduling loop needs to start from this match instead
// of walking the query again (MatchState: where the match ended, the run that position lies in, the next token).
struct alignas(32) MatchState {
    long long pos;        // pool index of the last matched token, -1 if nothing matched
    long long chain_end;  // end of the contiguous pool run `pos` lies in (trees with a budget: the node `pos` lies in)
    int32_t m;            // match length
    int32_t ntok;         // the query token right after the match (0 if the whole query matched)
    unsigned long long tag;   // which match call wrote this record
};
static_assert(sizeof(MatchState) == sizeof(klpm_match_state), "klpm_match_state is the ABI's view of MatchState");

template <bool STATE>
__global__ void __launch_bounds__(256, KLPM_MATCH_MIN_BLOCKS)
match_chain_kernel(TreeDev T, const int32_t* __restrict__ qtok, const int64_t* __restrict__ qoff, int32_t nq,
                   const int32_t* __restrict__ perm, int32_t* __restrict__ mlen, int32_t* __restrict__ tnode,
                   int32_t* __restrict__ toff, MatchState* __restrict__ state, unsigned long long tag,
                   unsigned long long* counter) {
    const int lane = threadIdx.x & 31;
    const bool want_node = tnode != nullptr || toff != nullptr;
    for (;;) {
        unsigned long long c = 0;
        if (lane == 0) c = atomicAdd(counter, 1ULL);
        c = __shfl_sync(FULL_MASK, c, 0);
        if (c >= (unsigned long long)nq) return;
        const int64_t i = perm ? (int64_t)__ldg(perm + c) : (int64_t)c;
        const int64_t lo = __ldg(qoff + i);
        int64_t len = __ldg(qoff + i + 1) - lo;
        if (len < 0 || len > 0x7fffffffLL) { if (lane == 0) set_status(T.st, RT_ERR_INVALID); len = 0; }
        int32_t node, off;
        int64_t pos = -1, cend = 0;
        const int32_t m = STATE ? walk_chain<true>(T, qtok + lo, (int32_t)len, want_node, &node, &off, &pos, &cend)
                                : walk_chain<false>(T, qtok + lo, (int32_t)len, want_node, &node, &off);
        if (lane == 0) {
            if (mlen) mlen[i] = m;
            if (tnode) tnode[i] = node;
            if (toff) toff[i] = off;
            if (STATE) {
                const int32_t ntok = m < (int32_t)len ? __ldg(qtok + lo + m) : 0;
                int4* dst = reinterpret_cast<int4*>(state + i);
                __stcg(dst, make_int4((int)(unsigned)(unsigned long long)pos, (int)(unsigned)((unsigned long long)pos >> 32),
                                      (int)(unsigned)(unsigned long long)cend, (int)(unsigned)((unsigned long long)cend >> 32)));
                __stcg(dst + 1, make_int4(m, ntok, (int)(unsigned)tag, (int)(unsigned)(tag >> 32)));
            }
        }
    }
}

// The order in which the batched match takes the queries: bucketed by first token (counting sort over a hash of
// it; the order inside a bucket is whatever the atomics give -- results do not depend on it).
#define KLPM_ORDER_BUCKETS 8192
__device__ __forceinline__ unsigned order_bucket(const int32_t* __restrict__ qtok, const int64_t* __restrict__ qoff, int32_t i) {
    const int64_t lo = __ldg(qoff + i);
    if (__ldg(qoff + i + 1) <= lo) return 0u;
    unsigned h = (unsigned)__ldg(qtok + lo) * 0x9E3779B1u;
    return h >> 19;                                         // 13 bits: KLPM_ORDER_BUCKETS
}
__global__ void order_hist_kernel(const int32_t* __restrict__ qtok, const int64_t* __restrict__ qoff, int32_t nq,
                                  unsigned* __restrict__ hist, unsigned short* __restrict__ bucket) {
    const int32_t i = blockIdx.x * blockDim.x + threadIdx.x;
    if (i >= nq) return;
    const unsigned b = order_bucket(qtok, qoff, i);
    bucket[i] = (unsigned short)b;
    atomicAdd(hist + b, 1u);
}
// hist[b] <- number of queries in buckets below b (one CTA of 1,024 threads, 8 buckets each)
__global__ void __launch_bounds__(1024) order_scan_kernel(unsigned* hist) {
    __shared__ unsigned s_w[32];
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    constexpr int PER = KLPM_ORDER_BUCKETS / 1024;
    unsigned v[PER], sum = 0;
#pragma unroll
    for (int j = 0; j < PER; ++j) { v[j] = hist[tid * PER + j]; sum += v[j]; }
    unsigned inc = sum;
#pragma unroll
    for (int d = 1; d < 32; d <<= 1) { const unsigned o = __shfl_up_sync(FULL_MASK, inc, d); if (lane >= d) inc += o; }
    if (lane == 31) s_w[warp] = inc;
    __syncthreads();
    if (warp == 0) {
        unsigned w = s_w[lane], wi = w;
#pragma unroll
        for (int d = 1; d < 32; d <<= 1) { const unsigned o = __shfl_up_sync(FULL_MASK, wi, d); if (lane >= d) wi += o; }
        s_w[lane] = wi - w;
    }
    __syncthreads();
    unsigned run = s_w[warp] + inc - sum;
#pragma unroll
    for (int j = 0; j < PER; ++j) { hist[tid * PER + j] = run; run += v[j]; }
}
__global__ void order_scatter_kernel(const unsigned short* __restrict__ bucket, int32_t nq, unsigned* __restrict__ cursor,
                                     int32_t* __restrict__ perm) {
    const int32_t i = blockIdx.x * blockDim.x + threadIdx.x;
    if (i >= nq) return;
    perm[atomicAdd(cursor + bucket[i], 1u)] = i;
}

// Trees with a budget (evicted children break the runs): hop by hop.
__global__ void __launch_bounds__(256)
match_batch_kernel(TreeDev T, const int32_t* __restrict__ qtok, const int64_t* __restrict__ qoff, int32_t nq,
                   const int32_t* __restrict__ perm, int32_t* __restrict__ mlen, int32_t* __restrict__ tnode,
                   int32_t* __restrict__ toff, MatchState* __restrict__ state, unsigned long long tag,
                   unsigned long long* counter) {
    const int lane = threadIdx.x & 31;
    for (;;) {
        unsigned long long c = 0;
        if (lane == 0) c = atomicAdd(counter, 1ULL);
        c = __shfl_sync(FULL_MASK, c, 0);
        if (c >= (unsigned long long)nq) return;
        const int64_t i = perm ? (int64_t)__ldg(perm + c) : (int64_t)c;
        const int64_t lo = __ldg(qoff + i), hi = __ldg(qoff + i + 1);
        int64_t len = hi - lo;
        if (len < 0 || len > 0x7fffffffLL) { if (lane == 0) set_status(T.st, RT_ERR_INVALID); len = 0; }
        Term t = walk<true>(T, qtok + lo, (int32_t)len);
        if (lane == 0) {
            if (mlen) mlen[i] = t.m;
            if (tnode) tnode[i] = t.node;
            if (toff) toff[i] = t.off;
            if (state) {
                MatchState r;
                // trees with a budget have no use for the run's end; the field carries the node the match ended in instead
                r.pos = t.pos; r.chain_end = t.node; r.m = t.m; r.ntok = t.m < (int32_t)len ? __ldg(qtok + lo + t.m) : 0; r.tag = tag;
                state[i] = r;
            }
        }
    }
}

// ------------------------------------------------------------------------------------------------
// sequential processing of prompts by one CTA: rt_insert and klpm_replay
// ------------------------------------------------------------------------------------------------
struct SeqArgs {
    const int32_t* tok; const int64_t* off; const int64_t* arrival; const int32_t* order;
    int32_t n;                       // prompts to process
    int32_t n_queries;               // prompts in the CSR arrays: entries of `order` must be below this
    long long c_num, c_den, start_tick;
    int32_t* new_tokens;             // rt_insert: indexed by position
    int32_t* uncached; int64_t* ttft; int64_t* completion;   // replay: indexed by query
};

__global__ void __launch_bounds__(1024)
sequential_kernel(TreeDev T, SeqArgs A) {
    __shared__ Term s_term;
    __shared__ InsertOut s_out;
    long long now = A.start_tick;
    for (int32_t k = 0; k < A.n; ++k) {
        const int32_t j = A.order ? __ldg(A.order + k) : k;
        if (j < 0 || j >= A.n_queries) {           // not a query: nothing of it is read or written (uniform over the CTA)
            if (threadIdx.x == 0) set_status(T.st, RT_ERR_INVALID, 108);
            return;
        }
        const int64_t lo = __ldg(A.off + j), hi = __ldg(A.off + j + 1);
        if (hi < lo || hi - lo > 0x7fffffffLL) {
            if (threadIdx.x == 0) set_status(T.st, RT_ERR_INVALID, 108);
            return;
        }
        const int32_t len = (int32_t)(hi - lo);
        const int32_t* x = A.tok + lo;
        if (threadIdx.x < 32) {
            Term t = walk<false>(T, x, len);
            if (threadIdx.x == 0) {
                s_term = t;
                insert_serial(T, x, len, t.m, t.node, &s_out);
                if (s_out.ok) {
                    int32_t unc = len - t.m;
                    if (A.new_tokens) A.new_tokens[k] = unc;
                    if (A.uncached) {
                        long long tj = __ldg(A.arrival + j);
                        long long begin = now > tj ? now : tj;
                        long long R = begin + (A.c_den + A.c_num * (long long)len) * (long long)unc;
                        A.uncached[j] = unc; A.ttft[j] = R - tj;
                        if (A.completion) A.completion[j] = R;
                        now = R;
                    }
                }
            }
        }
        __syncthreads();
        if (!s_out.ok) return;
        const int32_t unc = s_out.unc, m = s_term.m;
        int32_t* dst = T.pool + s_out.leaf_off;
        for (int32_t i = threadIdx.x; i < unc; i += blockDim.x) dst[i] = __ldg(x + m + i);
        __threadfence();
        __syncthreads();
    }
}

// ------------------------------------------------------------------------------------------------
// klpm_select: one decision as a pure function
// ------------------------------------------------------------------------------------------------
struct Cand { int32_t m; int32_t idx; long long t; };   // idx < 0 = none

__device__ __forceinline__ bool better_lpm(const Cand& a, const Cand& b) {      // a beats b
    if (b.idx < 0) return a.idx >= 0;
    if (a.idx < 0) return false;
    if (a.m != b.m) return a.m > b.m;
    if (a.t != b.t) return a.t < b.t;
    return a.idx < b.idx;
}
__device__ __forceinline__ bool better_fcfs(const Cand& a, const Cand& b) {
    if (b.idx < 0) return a.idx >= 0;
    if (a.idx < 0) return false;
    if (a.t != b.t) return a.t < b.t;
    return a.idx < b.idx;
}
template <bool LPM> __device__ __forceinline__ Cand cand_best(Cand a, Cand b) {
    return (LPM ? better_lpm(b, a) : better_fcfs(b, a)) ? b : a;
}
template <bool LPM> __device__ __forceinline__ Cand warp_best(Cand c) {
#pragma unroll
    for (int d = 16; d > 0; d >>= 1) {
        Cand o;
        o.m = __shfl_xor_sync(FULL_MASK, c.m, d);
        o.idx = __shfl_xor_sync(FULL_MASK, c.idx, d);
        o.t = __shfl_xor_sync(FULL_MASK, c.t, d);
        c = cand_best<LPM>(c, o);
    }
    return c;
}
template <bool LPM> __device__ Cand block_best(Cand c, Cand* smem /*32*/) {
    c = warp_best<LPM>(c);
    const int lane = threadIdx.x & 31, w = threadIdx.x >> 5, nw = (blockDim.x + 31) >> 5;
    if (lane == 0) smem[w] = c;
    __syncthreads();
    Cand r; r.m = 0; r.idx = -1; r.t = 0;
    if (w == 0) {
        if (lane < nw) r = smem[lane];
        r = warp_best<LPM>(r);
    }
    return r;   // valid in warp 0
}

struct SelectScratch { Cand partial[1024]; unsigned int ticket; };

template <bool LPM>
__global__ void __launch_bounds__(512)
select_kernel(const int32_t* __restrict__ mlen, const int64_t* __restrict__ arrival, const uint8_t* __restrict__ waiting,
              int32_t nq, int32_t* pick, SelectScratch* sc) {
    __shared__ Cand s_c[32];
    __shared__ bool s_last;
    Cand best; best.m = 0; best.idx = -1; best.t = 0;
    for (int64_t i = (int64_t)blockIdx.x * blockDim.x + threadIdx.x; i < nq; i += (int64_t)gridDim.x * blockDim.x) {
        if (__ldg(waiting + i)) {
            Cand c; c.m = LPM ? __ldg(mlen + i) : 0; c.idx = (int32_t)i; c.t = __ldg(arrival + i);
            best = cand_best<LPM>(best, c);
        }
    }
    best = block_best<LPM>(best, s_c);
    if (threadIdx.x == 0) {
        sc->partial[blockIdx.x] = best;
        __threadfence();
        unsigned t = atomicAdd(&sc->ticket, 1u);
        s_last = (t == gridDim.x - 1);
    }
    __syncthreads();
    if (!s_last) return;
    __threadfence();
    Cand c; c.m = 0; c.idx = -1; c.t = 0;
    for (int b = threadIdx.x; b < (int)gridDim.x; b += blockDim.x) {
        Cand o;
        o.m = __ldcg(&sc->partial[b].m); o.idx = __ldcg(&sc->partial[b].idx); o.t = __ldcg(&sc->partial[b].t);
        c = cand_best<LPM>(c, o);
    }
    __syncthreads();
    c = block_best<LPM>(c, s_c);
    if (threadIdx.x == 0) { *pick = c.idx; sc->ticket = 0; }
}

// ------------------------------------------------------------------------------------------------
// klpm_select_topk: the kk best longest-match candidates of one queue snapshot, best first.
// The j-th best is the best element strictly worse than the (j-1)-th in the total order
// (match desc, arrival asc, index asc), so no element is ever marked as taken: each CTA extracts its own
// kk best by kk passes over its slice, and the last CTA to finish merges the per-CTA lists the same way.
// ------------------------------------------------------------------------------------------------
#define KLPM_TOPK_MAX 64
#define KLPM_TOPK_BLOCKS 128
struct TopkScratch { Cand cand[KLPM_TOPK_BLOCKS * KLPM_TOPK_MAX]; unsigned int ticket; };

__global__ void __launch_bounds__(512)
select_topk_kernel(const int32_t* __restrict__ mlen, const int64_t* __restrict__ arrival, const uint8_t* __restrict__ waiting,
                   int32_t nq, int32_t kk, int32_t* out, TopkScratch* sc) {
    __shared__ Cand s_c[32];
    __shared__ Cand s_prev;
    __shared__ bool s_last;
    Cand prev; prev.m = 0; prev.idx = -1; prev.t = 0;          // idx < 0: no bound yet
    for (int j = 0; j < kk; ++j) {
        Cand best; best.m = 0; best.idx = -1; best.t = 0;
        for (int64_t i = (int64_t)blockIdx.x * blockDim.x + threadIdx.x; i < nq; i += (int64_t)gridDim.x * blockDim.x) {
            if (__ldg(waiting + i)) {
                Cand c; c.m = __ldg(mlen + i); c.idx = (int32_t)i; c.t = __ldg(arrival + i);
                if (prev.idx < 0 || better_lpm(prev, c)) best = cand_best<true>(best, c);
            }
        }
        best = block_best<true>(best, s_c);
        if (threadIdx.x == 0) { s_prev = best; sc->cand[blockIdx.x * KLPM_TOPK_MAX + j] = best; }
        __syncthreads();
        prev = s_prev;
        __syncthreads();
        if (prev.idx < 0) {                                     // slice exhausted: pad the rest
            if (threadIdx.x == 0) for (int r = j + 1; r < kk; ++r) sc->cand[blockIdx.x * KLPM_TOPK_MAX + r] = prev;
            break;
        }
    }
    if (threadIdx.x == 0) {
        __threadfence();
        s_last = atomicAdd(&sc->ticket, 1u) == gridDim.x - 1;
    }
    __syncthreads();
    if (!s_last) return;
    __threadfence();
    prev.m = 0; prev.idx = -1; prev.t = 0;
    bool done = false;
    for (int j = 0; j < kk; ++j) {
        Cand best; best.m = 0; best.idx = -1; best.t = 0;
        if (!done) {
            for (int e = threadIdx.x; e < (int)gridDim.x * kk; e += blockDim.x) {
                const Cand* src = &sc->cand[(e / kk) * KLPM_TOPK_MAX + (e % kk)];
                Cand c; c.m = __ldcg(&src->m); c.idx = __ldcg(&src->idx); c.t = __ldcg(&src->t);
                if (c.idx >= 0 && (prev.idx < 0 || better_lpm(prev, c))) best = cand_best<true>(best, c);
            }
        }
        __syncthreads();
        best = block_best<true>(best, s_c);
        if (threadIdx.x == 0) { s_prev = best; out[j] = best.idx; }
        __syncthreads();
        if (s_prev.idx < 0) done = true; else prev = s_prev;
        __syncthreads();
    }
    if (threadIdx.x == 0) sc->ticket = 0;
}

// ------------------------------------------------------------------------------------------------
// klpm_select_noalloc: the same decision as klpm_select, with the per-CTA partial results kept in a
// fixed array that is part of the library image instead of memory obtained from cudaMalloc.
// ------------------------------------------------------------------------------------------------
#define KLPM_SELECT_NOALLOC_BLOCKS 256
struct StaticSelectScratch { Cand partial[KLPM_SELECT_NOALLOC_BLOCKS]; unsigned int ticket; };
// 4 KiB + one counter per GPU that loads the library, held until the process exits.
static __device__ __align__(256) unsigned char g_select_static[sizeof(StaticSelectScratch)];

template <bool LPM>
__global__ void __launch_bounds__(512)
select_static_kernel(const int32_t* __restrict__ mlen, const int64_t* __restrict__ arrival, const uint8_t* __restrict__ waiting,
                     int32_t nq, int32_t* pick, StaticSelectScratch* sc) {
    __shared__ Cand s_c[32];
    __shared__ bool s_last;
    Cand best; best.m = 0; best.idx = -1; best.t = 0;
    for (int64_t i = (int64_t)blockIdx.x * blockDim.x + threadIdx.x; i < nq; i += (int64_t)gridDim.x * blockDim.x) {
        if (__ldg(waiting + i)) {
            Cand c; c.m = LPM ? __ldg(mlen + i) : 0; c.idx = (int32_t)i; c.t = __ldg(arrival + i);
            best = cand_best<LPM>(best, c);
        }
    }
    best = block_best<LPM>(best, s_c);
    if (threadIdx.x == 0) {
        sc->partial[blockIdx.x] = best;
        __threadfence();
        s_last = atomicAdd(&sc->ticket, 1u) == gridDim.x - 1;
    }
    __syncthreads();
    if (!s_last) return;
    __threadfence();
    Cand c; c.m = 0; c.idx = -1; c.t = 0;
    for (int b = threadIdx.x; b < (int)gridDim.x; b += blockDim.x) {
        Cand o;
        o.m = __ldcg(&sc->partial[b].m); o.idx = __ldcg(&sc->partial[b].idx); o.t = __ldcg(&sc->partial[b].t);
        c = cand_best<LPM>(c, o);
    }
    __syncthreads();
    c = block_best<LPM>(c, s_c);
    if (threadIdx.x == 0) *pick = c.idx;
}

// ------------------------------------------------------------------------------------------------
// klpm_run, one decision at a time on the tree itself: the whole loop as one cooperative kernel.
// Trees with a budget take this loop (eviction can shorten matches, so match lengths are kept against
// the tree as it changes); trees without one take the grouped loop further down.
//
// Slots are the queries ordered by (arrival, index).  Per decision c:
//   phase A (every CTA): bring the match state of the waiting slots up to date -- walk newly arrived
//     queries, drop queries out of evicted leaves, extend the queries that were tied with the prompt
//     processed last into its new leaf -- and reduce the keys (match << 32 | ~slot) to one per CTA;
//   phase B (CTA 0): pick (oldest waiting slot or largest key), charge by Definition 2, store the prompt.
// The two phases hand over through two monotone counters in global memory (`arrive`: CTAs that finished
// phase A; `seq`: decisions completed), and what phase A needs to know about the last decision travels
// in one broadcast record.  While the kernel runs only CTA 0 mutates the tree; it keeps the tree's
// counters in shared memory and writes them back at the end.
// ------------------------------------------------------------------------------------------------
struct RunBcast {
    long long now;            // completion time of the last processed query
    long long head;           // first slot not yet processed
    long long admitted;       // slots < admitted have a match state
    long long last_pos;       // position (pool index of last matched token) of the last processed prompt, before it was stored
    long long last_leaf_off;  // pool offset of the leaf it appended
    int32_t evicted;          // the last decision evicted something
    int32_t last_valid;       // the last decision appended a leaf
    int32_t last_q, last_m, last_len, last_leaf;
    int32_t abort;
    int32_t last_xm;          // first uncached token of the last processed prompt
};
struct RunSync { unsigned long long arrive; unsigned long long seq; };

struct RunArgs {
    const int32_t* tok; const int64_t* off; const int64_t* arrival;
    int32_t n;
    int32_t policy, k;
    long long c_num, c_den, start_tick;
    int32_t* order; int32_t* uncached; int64_t* ttft; int64_t* completion;
    // scratch (library-owned)
    int32_t* ord;          // slot -> query index, by (arrival, index)
    long long* sorted_t;   // slot -> arrival
    long long* soff;       // slot -> offset of the query's first token
    int32_t* slen;         // slot -> query length
    int32_t* m;            // slot -> current match length; -1 once processed
    int32_t* hint;         // slot -> node at or below the node where the match ends
    long long* pos;        // slot -> pool index of the last matched token (-1 = root)
    int32_t* ntok;         // slot -> the query token right after its match (meaningful while m < length)
    const int32_t* prank;  // slot -> rank of the slot by (tie priority, slot); null = ties go to the lower slot
    const int32_t* pinv;   // that rank -> slot
    int32_t score_mode;    // 0: score = match length; 1: score = floor(match * 2^31 / length)
    unsigned long long* partial;   // per CTA best key
    RunBcast* bc;
    RunSync* sy;
    long long wait_limit_ns;       // limit of every hand-over wait
};

#define KLPM_RUN_THREADS 512
#define KLPM_RUN_SLOTS 4          // slots per thread whose state is loaded together
#ifndef KLPM_RUN_SPT
#define KLPM_RUN_SPT 2            // slots per scanner thread the grid is sized for
#endif
#define KLPM_WAIT_LIMIT_NS 5000000000LL      // default limit of a hand-over wait: 5 s on the device's nanosecond timer

// Thread 0 of the CTA polls *p until it reaches target, then the CTA learns whether to go on.  The wait is
// bounded: after limit_ns (checked every 4,096 polls; a limit of 0 gives up at the first poll that fails) the
// status word gets RT_ERR_LIMIT, every CTA is told to leave, and this one returns false.
__device__ bool run_wait(volatile unsigned long long* p, unsigned long long target, RunBcast* bc, TreeState* st, long long limit_ns) {
    __shared__ int s_go;
    if (threadIdx.x == 0) {
        int go = 1;
        unsigned long long spins = 0, t0 = 0;
        while (*p < target) {
            if ((++spins & 4095ULL) == 0 || limit_ns == 0) {
                unsigned long long now;
                asm volatile("mov.u64 %0, %globaltimer;" : "=l"(now));
                if (t0 == 0) t0 = now;
                if (limit_ns == 0 || now - t0 > (unsigned long long)limit_ns || spins > (1ULL << 40)) {
                    set_status(st, RT_ERR_LIMIT, 102); *(volatile int32_t*)&bc->abort = 1; go = 0; break;
                }
            }
        }
        __threadfence();
        if (*(volatile int32_t*)&bc->abort) go = 0;
        s_go = go;
    }
    __syncthreads();
    const bool go = s_go != 0;
    __syncthreads();
    return go;
}

// Time at which the next pick is made and the number of slots that have arrived by then (one thread).
// Everything below `admitted` has arrived already, so the search gallops from there.
__device__ void run_bound(const RunArgs& A, const RunBcast& b, long long* adm_new, long long* now_out) {
    long long now = b.now;
    if (b.head >= b.admitted && b.head < A.n) {   // nobody waiting: idle until the next arrival
        const long long th = __ldg(A.sorted_t + b.head);
        if (th > now) now = th;
    }
    long long lo = b.admitted > b.head ? b.admitted : b.head, hi = A.n;
    if (lo < hi && __ldg(A.sorted_t + lo) <= now) {
        long long step = 1;
        ++lo;
        while (lo + step <= hi && __ldg(A.sorted_t + lo + step - 1) <= now) { lo += step; step <<= 1; }
        if (lo + step < hi) hi = lo + step;
        while (lo < hi) { const long long mid = (lo + hi) >> 1; if (__ldg(A.sorted_t + mid) <= now) lo = mid + 1; else hi = mid; }
    }
    *adm_new = lo; *now_out = now;
}

// Phase A for one CTA of the `nscan` scanning CTAs: returns (in warp lanes) this thread's best key.
__device__ unsigned long long run_scan(const TreeDev& T, const RunArgs& A, const RunBcast& bc, long long adm_new,
                                       unsigned scan_id, unsigned nscan) {
    const int lane = threadIdx.x & 31;
    const long long TT = (long long)nscan * blockDim.x;
    const long long gtid = (long long)scan_id * blockDim.x + threadIdx.x;
    const long long head = bc.head, admitted = bc.admitted;
    const int evicted = bc.evicted, last_valid = bc.last_valid;
    const int32_t last_m = bc.last_m, last_len = bc.last_len, last_leaf = bc.last_leaf;
    const long long last_pos = bc.last_pos, last_leaf_off = bc.last_leaf_off;
    const int32_t last_xm = bc.last_xm;
    const int32_t* last_x = last_valid ? A.tok + __ldg(A.off + bc.last_q) : nullptr;
    unsigned long long best = 0;
    for (long long base = (head / TT) * TT; base < adm_new; base += TT * KLPM_RUN_SLOTS) {
        int32_t mm[KLPM_RUN_SLOTS], nn[KLPM_RUN_SLOTS];
        long long pp[KLPM_RUN_SLOTS];
#pragma unroll
        for (int u = 0; u < KLPM_RUN_SLOTS; ++u) {
            const long long r = base + u * TT + gtid;
            const bool have = r >= head && r < admitted && r < adm_new;
            mm[u] = have ? __ldcg(A.m + r) : -1;
            pp[u] = have ? __ldcg(A.pos + r) : -1;
            nn[u] = have ? __ldcg(A.ntok + r) : 0;
        }
#pragma unroll
        for (int u = 0; u < KLPM_RUN_SLOTS; ++u) {
            if (base + u * TT >= adm_new) break;                               // warp-uniform
            const long long r = base + u * TT + gtid;
            const bool fresh = r >= head && r >= admitted && r < adm_new;
            int32_t m = mm[u], hint = 0, ntok = nn[u];
            long long pos = pp[u];
            bool dirty = false;
            unsigned wm = __ballot_sync(FULL_MASK, fresh);
            if (wm) {                                  // newly arrived queries: full walk, one warp each
                const int32_t* q = nullptr; int32_t qlen = 0;
                if (fresh) { qlen = __ldg(A.slen + r); q = A.tok + __ldg(A.soff + r); }
                while (wm) {
                    const int src = __ffs(wm) - 1; wm &= wm - 1;
                    const int32_t* qq = (const int32_t*)__shfl_sync(FULL_MASK, (unsigned long long)q, src);
                    const int32_t ql = __shfl_sync(FULL_MASK, qlen, src);
                    Term t = walk<false>(T, qq, ql);
                    if (lane == src) { m = t.m; hint = t.node; pos = t.pos; ntok = t.m < ql ? __ldg(qq + t.m) : 0; dirty = true; }
                }
            }
            const bool waiting = fresh || m >= 0;
            if (waiting && !fresh && evicted) {        // drop out of evicted leaves
                hint = __ldcg(A.hint + r);
                int32_t a = hint;
                const int32_t m0 = m;
                while (a != 0) {
                    const bool dead = __ldcg(T.dead + a) != 0;
                    const int32_t ds = __ldcg(T.depth_start + a);
                    if (dead) { if (ds < m) m = ds; }
                    else if (m > ds) break;
                    a = __ldcg(T.parent + a);
                }
                if (a != hint || m != m0) {
                    hint = a;
                    pos = a == 0 ? -1 : __ldcg(T.span_off + a) + (m - __ldcg(T.depth_start + a)) - 1;
                    if (m != m0) ntok = m < __ldg(A.slen + r) ? __ldg(A.tok + __ldg(A.soff + r) + m) : 0;
                    dirty = true;
                } else {
                    hint = -1;                          // unchanged: do not rewrite
                }
            }
            // tied with the prompt processed last: it may now match into that prompt's new leaf
            bool cmp = false;
            const int32_t* q = nullptr; int32_t qlen = 0;
            if (waiting && !fresh && last_valid && pos == last_pos && m == last_m && ntok == last_xm) {
                qlen = __ldg(A.slen + r);
                q = A.tok + __ldg(A.soff + r);
                cmp = m < qlen;
            }
            unsigned cm = __ballot_sync(FULL_MASK, cmp);
            while (cm) {
                const int src = __ffs(cm) - 1; cm &= cm - 1;
                const int32_t* qq = (const int32_t*)__shfl_sync(FULL_MASK, (unsigned long long)q, src);
                const int32_t ql = __shfl_sync(FULL_MASK, qlen, src);
                const int32_t lim = (ql < last_len ? ql : last_len) - last_m;
                const int32_t e = first_mismatch<true>(qq + last_m, last_x + last_m, lim);
                if (lane == src) {
                    m = last_m + e; hint = last_leaf; pos = last_leaf_off + e - 1;
                    ntok = m < ql ? __ldg(qq + m) : 0;
                    dirty = true;
                }
            }
            if (waiting) {
                if (dirty) { A.m[r] = m; A.pos[r] = pos; A.ntok[r] = ntok; if (hint >= 0) A.hint[r] = hint; }
                unsigned hi = (unsigned)m;
                if (A.score_mode == 1) {
                    const int32_t ql = __ldg(A.slen + r);
                    hi = ql > 0 ? (unsigned)(((unsigned long long)(unsigned)m << 31) / (unsigned)ql) : 0u;
                }
                const unsigned lo = A.prank ? (unsigned)__ldg(A.prank + r) : (unsigned)r;
                const unsigned long long key = ((unsigned long long)hi << 32) | (0xffffffffu - lo);
                if (key > best) best = key;
            }
        }
    }
    return best;
}

__device__ __forceinline__ unsigned long long warp_max64(unsigned long long v) {
#pragma unroll
    for (int d = 16; d > 0; d >>= 1) {
        const unsigned long long o = __shfl_xor_sync(FULL_MASK, v, d);
        if (o > v) v = o;
    }
    return v;
}

// CTA 0 is the sequencer (picks, charges, mutates the tree); CTAs 1..G-1 scan.  With a single CTA it does both.
// Without a budget, and when the next decision admits no new arrivals, the sequencer publishes its pick --
// including the id and pool offset its new leaf is going to get, which follow from the tree's counters --
// before it performs the insertion, so the scanners refresh the waiting queue for the next decision while
// the tree is being updated (they only read query tokens and their own slots' state then).
__global__ void __launch_bounds__(KLPM_RUN_THREADS)
run_kernel(TreeDev T, RunArgs A) {
    __shared__ unsigned long long s_red[KLPM_RUN_THREADS / 32];
    __shared__ long long s_bound[2];      // slots admitted by this decision, time at which the pick is made
    __shared__ InsertOut s_out;
    __shared__ int32_t s_j[2];            // match length and length of the picked prompt
    __shared__ const int32_t* s_x;
    __shared__ TreeState s_st;            // CTA 0: the tree's counters while the kernel runs
    __shared__ RunBcast s_bc;
    __shared__ int s_flag[2];             // CTA 0: publish-before-insert, predicted leaf
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    const unsigned G = gridDim.x;
    const unsigned nscan = G > 1 ? G - 1 : 1;
    TreeState* const gst = T.st;

    if (blockIdx.x != 0) {
        // ------------------------------------------------------------ scanners
        for (long long c = 0; c < A.n; ++c) {
            if (!run_wait(&A.sy->seq, (unsigned long long)c, A.bc, gst, A.wait_limit_ns)) return;
            if (threadIdx.x == 0) {
                RunBcast b;
                const long long* src = reinterpret_cast<const long long*>(A.bc);
                long long* dst = reinterpret_cast<long long*>(&b);
#pragma unroll
                for (int i = 0; i < (int)(sizeof(RunBcast) / 8); ++i) dst[i] = __ldcg(src + i);
                s_bc = b;
                run_bound(A, b, &s_bound[0], &s_bound[1]);
            }
            __syncthreads();
            unsigned long long best = warp_max64(run_scan(T, A, s_bc, s_bound[0], blockIdx.x - 1, nscan));
            if (lane == 0) s_red[warp] = best;
            __syncthreads();
            if (threadIdx.x == 0) {
                unsigned long long b = 0;
                for (int w = 0; w < (int)(blockDim.x >> 5); ++w) if (s_red[w] > b) b = s_red[w];
                A.partial[blockIdx.x - 1] = b;
                __threadfence();
                atomicAdd(&A.sy->arrive, 1ULL);
            }
        }
        return;
    }

    // ---------------------------------------------------------------- sequencer (CTA 0)
    TreeDev T0 = T;                        // its view of the tree: counters in shared memory
    T0.st = &s_st;
    if (threadIdx.x == 0) {
        s_st = *gst;
        RunBcast b;
        const long long* src = reinterpret_cast<const long long*>(A.bc);
        long long* dst = reinterpret_cast<long long*>(&b);
#pragma unroll
        for (int i = 0; i < (int)(sizeof(RunBcast) / 8); ++i) dst[i] = __ldcg(src + i);
        s_bc = b;
    }
    __syncthreads();
    bool ok = true;
    for (long long c = 0; c < A.n && ok; ++c) {
        if (threadIdx.x == 0) run_bound(A, s_bc, &s_bound[0], &s_bound[1]);
        __syncthreads();
        const long long head = s_bc.head, adm_new = s_bound[0];
        // The queries that arrive next will be walked from the root by a single warp while everybody waits: bring
        // their tokens into L2 now (slots are in arrival order, so these are known; a hint only).
        for (long long r = adm_new; r < adm_new + 2 && r < A.n; ++r) {
            const int32_t* q = A.tok + __ldg(A.soff + r);
            const int32_t qlen = __ldg(A.slen + r);
            for (int32_t i = threadIdx.x * 32; i < qlen; i += blockDim.x * 32) asm volatile("prefetch.global.L2 [%0];" ::"l"(q + i));
        }
        unsigned long long b = 0;
        if (G == 1) {
            unsigned long long best = warp_max64(run_scan(T, A, s_bc, adm_new, 0, 1));
            if (lane == 0) s_red[warp] = best;
            __syncthreads();
            if (warp == 0) b = warp_max64(lane < (int)(blockDim.x >> 5) ? s_red[lane] : 0ULL);
        } else {
            if (!run_wait(&A.sy->arrive, (unsigned long long)(c + 1) * nscan, A.bc, gst, A.wait_limit_ns)) { ok = false; break; }
            if (warp == 0) {
                for (unsigned g = lane; g < nscan; g += 32) { const unsigned long long o = __ldcg(A.partial + g); if (o > b) b = o; }
                b = warp_max64(b);
            }
        }
        // ---- pick (warp 0; lane 0 decides), charge by Definition 2
        if (warp == 0) {
            const bool fcfs_turn = A.policy == KLPM_POLICY_FCFS || (A.policy == KLPM_POLICY_KLPM && (c % A.k) == 0);
            long long slot = head;
            if (!fcfs_turn) {
                const unsigned rk = 0xffffffffu - (unsigned)(b & 0xffffffffu);
                slot = A.pinv ? (long long)__ldg(A.pinv + rk) : (long long)rk;
            }
            const int32_t qi = __ldg(A.ord + slot);
            const int32_t m = __ldcg(A.m + slot);
            const int32_t hint = __ldcg(A.hint + slot);
            const long long pos = __ldcg(A.pos + slot);
            const int32_t ntok = __ldcg(A.ntok + slot);
            const int32_t len = __ldg(A.slen + slot);
            const long long tj = __ldg(A.sorted_t + slot);
            const int32_t* x = A.tok + __ldg(A.soff + slot);
            // where the cached part ends, and what the insertion is going to allocate
            int32_t a = hint;
            int32_t a_ds = T.depth_start[a], a_sl = T.span_len[a], a_par = T.parent[a], a_ft = T.first_tok[a];   // side by side
            const int32_t below = __ldcg(T.pool + (pos + 1));       // the pool token under the cut, if there is a cut
            while (a != 0 && m <= a_ds) {
                a = a_par;
                a_ds = T.depth_start[a]; a_sl = T.span_len[a]; a_par = T.parent[a]; a_ft = T.first_tok[a];
            }
            const int32_t o = a == 0 ? 0 : m - a_ds;
            const bool mid = a != 0 && o < a_sl;
            const int32_t unc = len - m;
            const int32_t leaf_pred = unc > 0 ? (int32_t)s_st.n_nodes + (mid ? 1 : 0) : -1;
            const long long leaf_off_pred = unc > 0 ? ((s_st.pool_used + 3) & ~3LL) + (m & 3) : 0;
            // Three lanes read, side by side, what the serial insertion would otherwise wait for one after
            // the other: the tokens that key its table operations, then the first slot each will probe.
            // The reads are issued here and collected after the pick has been published.
            int32_t v = 0;
            if (lane == 0 && unc > 0) v = ntok;
            if (lane == 1 && mid) v = below;
            if (lane == 2 && mid) v = a_ft;
            unsigned long long seen = 0;
            {
                const int32_t end = mid ? (int32_t)s_st.n_nodes : a;
                unsigned long long key = 0;
                bool want = false;
                if (lane == 0) { key = make_key(end, v); want = unc > 0; }
                if (lane == 1) { key = make_key(end, v); want = mid; }
                if (lane == 2) { key = make_key(a_par, v); want = mid; }
                if (want) seen = __ldcg(&T.table[hash_key(key) & T.table_mask].key);
                for (int32_t i = lane * 32; i < unc; i += 32 * 32) asm volatile("prefetch.global.L2 [%0];" ::"l"(x + m + i));
            }
            if (lane == 0) {
                s_j[0] = m; s_j[1] = len; s_x = x;
                const long long now = s_bound[1];
                const long long begin = now > tj ? now : tj;
                const long long R = begin + (A.c_den + A.c_num * (long long)len) * (long long)unc;
                A.m[slot] = -1;
                long long h = head;
                if (slot == head) while (h < A.n && (h == slot || (h < adm_new && __ldcg(A.m + h) < 0))) ++h;
                RunBcast nb = s_bc;
                nb.head = h; nb.now = R; nb.admitted = adm_new;
                nb.evicted = 0;
                nb.last_valid = unc > 0; nb.last_q = qi; nb.last_m = m; nb.last_len = len;
                nb.last_leaf = leaf_pred; nb.last_pos = pos; nb.last_leaf_off = leaf_off_pred; nb.last_xm = ntok;
                s_bc = nb;
                // may the scanners start on the next decision while the tree is being updated?
                long long adm_next, now_next;
                run_bound(A, nb, &adm_next, &now_next);
                const int early = (G > 1 && T.budget == 0 && adm_next == adm_new && c + 1 < A.n) ? 1 : 0;
                s_flag[0] = early; s_flag[1] = leaf_pred;
                if (early) {
                    *A.bc = nb;
                    __threadfence();
                    atomicExch(&A.sy->seq, (unsigned long long)(c + 1));
                }
                A.order[c] = qi; A.uncached[qi] = unc; A.ttft[qi] = R - tj;
                if (A.completion) A.completion[qi] = R;
            }
            InsertPre pre;
            pre.xm = __shfl_sync(FULL_MASK, v, 0); pre.pt = __shfl_sync(FULL_MASK, v, 1); pre.ft = __shfl_sync(FULL_MASK, v, 2);
            pre.k_leaf = __shfl_sync(FULL_MASK, seen, 0); pre.k_low = __shfl_sync(FULL_MASK, seen, 1); pre.k_par = __shfl_sync(FULL_MASK, seen, 2);
            if (lane == 0) {
                insert_serial(T0, x, len, m, hint, &s_out, &pre);
                if (s_out.ok && (s_out.leaf != leaf_pred || (unc > 0 && s_out.leaf_off != leaf_off_pred))) {
                    set_status(&s_st, RT_ERR_LIMIT, 103);           // cannot happen: the prediction repeats the allocation rule
                    s_out.ok = 0;
                }
            }
        }
        __syncthreads();
        if (!s_out.ok) { ok = false; break; }
        {
            const int32_t unc = s_out.unc, m = s_j[0];
            const int32_t* x = s_x;
            int32_t* dst = T.pool + s_out.leaf_off;
            for (int32_t i = threadIdx.x; i < unc; i += blockDim.x) dst[i] = __ldg(x + m + i);
        }
        if (!s_flag[0]) __threadfence();       // published next: others may walk the tree (the early mode's readers never touch it)
        __syncthreads();
        if (threadIdx.x == 0 && !s_flag[0]) {
            s_bc.evicted = s_out.evicted;
            if (G > 1 && c + 1 < A.n) {
                *A.bc = s_bc;
                __threadfence();
                atomicExch(&A.sy->seq, (unsigned long long)(c + 1));
            }
        }
        __syncthreads();
    }
    __syncthreads();
    if (threadIdx.x == 0) {
        const int st_global = *(volatile int*)&gst->status;
        TreeState out = s_st;
        if (out.status == 0) { out.status = st_global; out.detail = *(volatile int*)&gst->detail; }
        *gst = out;
        if (!ok) *(volatile int32_t*)&A.bc->abort = 1;
        __threadfence();
        atomicExch(&A.sy->seq, (unsigned long long)A.n + 1);      // releases anybody still waiting
    }
}

// ------------------------------------------------------------------------------------------------
// klpm_run on a tree without a budget: the grouped loop.
//
// Without eviction the match length of a query only ever grows, and it grows exactly when a prompt is
// processed whose own match ended at the same tree position and continues with the same token
// (otherwise the processed prompt shares no more with the query than the tree already did).  So the loop
// needs no tree at all:
//   * every query -- arrived or not -- is matched once against the tree as it stands (one warp per query,
//     streaming along contiguous pool runs), which gives its match length m, the position `pos` where the
//     match ends (pool index of the last matched token) and the query token `ntok` that follows;
//   * queries with the same (pos, ntok) form a group, held as a contiguous run of a member array
//     (a bitonic sort by a 62-bit hash of the pair puts equal pairs side by side; a hash collision only
//     puts two groups into one run, and members are checked against (pos, ntok) before they are touched);
//   * when a prompt is processed its group is dissolved: every member is compared with the prompt's
//     uncached tokens, gets its new m, a position inside the prompt's new leaf and its next token, and the
//     members are regrouped by their new pairs inside the run they already occupy (they never need more
//     room: the processed query leaves).  A query in a group of one costs nothing.  Leaves created by the
//     loop get positions from a counter that starts above every real pool index;
//   * while arrivals are pending, the longest-match pick is the root of a tournament over the keys
//     (score << 32 | ~rank) of the arrived queries: 32-ary, leaves in global memory, every level above in shared
//     memory; once everybody has arrived it is the next entry of a list of all keys sorted before the loop, and the
//     tournament only holds the queries whose key has changed since (see fast_run_kernel);
//   * the oldest-first pick is a cursor over a bitmap of processed slots.
// One CTA runs the whole loop: warp 0 is the sequencer, the other warps wait at a named barrier and join
// for work that is worth sharing (a large group, a large batch of arrivals).  There is no wait on another
// CTA anywhere.  The processed prompts are stored in the tree afterwards, all at once, by the concurrent
// bulk insertion: the set of node boundaries does not depend on the order of insertion.
// ------------------------------------------------------------------------------------------------
struct alignas(32) FDyn {     // what the loop changes, one 32-byte sector per slot
    long long pos;            // pool index (real or virtual) of the last matched token, -1 at the root
    int32_t m;                // match length; -1 once processed
    int32_t ntok;             // query token right after the match (meaningful while m < length)
    int32_t gstart, gcount;   // the slot's group: run [gstart, gstart + gcount) of the member array
    int32_t hint;             // trees with a budget: a node at or below the node the match ends in (walk up while m <= depth_start)
    int32_t pad;
};
struct alignas(32) FStat {    // constant during the loop; the first 16 bytes are all that charging a pick needs
    long long t;              // arrival
    int32_t len;
    int32_t ord;              // query index
    long long soff;           // offset of the query's first token
    int32_t rank;             // low key bits: rank by (tie priority, slot), or the slot itself
    int32_t pad;
};

struct FastPost {
    int32_t c0; int32_t pad; long long now0;    // first decision made in list mode; the time it was made at
    // what the loop did (rt_debug_counters): careful steps, dissolves by the whole CTA, fallback scans, slots that fell
    // back, evictions; cycles spent in tree updates, fallback scans, dissolves; list mode: CTA-wide batches tried and
    // committed, decisions they made, warp-wide steps, decisions they made, decisions made one at a time; cycles in
    // CTA-wide attempts and in warp-wide attempts
    long long counters[16];
};

struct FastArgs {
    const int32_t* tok;
    int32_t n;
    int32_t policy, k, score_mode;
    long long c_num, c_den, start_tick;
    int32_t* order; int32_t* uncached; int64_t* ttft; int64_t* completion;
    FDyn* dyn; FStat* stat;
    unsigned long long* key;      // slot -> key it has (or will have once arrived); 0 once processed
    int32_t* mem;                 // member array
    const int32_t* pinv;          // rank -> slot, or null
    long long* gh; int32_t* gidx; // group hashes and slots (sorted before the loop; scratch for large groups inside it)
    unsigned int* done;           // bitmap of processed slots (used when it does not fit in shared memory)
    long long vbase;              // first virtual pool index
    int32_t lb_shift;             // log2 of the number of slots per tournament leaf block
    int32_t nb;                   // number of leaf blocks
    int32_t done_in_smem;
    int32_t list_mode;            // the list mode of the loop can be used (trees without a budget)
    unsigned int* gbits;          // bitmap of slots whose group has more than one member, as the loop starts (and throughout, if the bitmaps stay in global memory)
    unsigned int* gskip;          // list mode with the bitmaps in global memory: slots the sorted list must pass over
    int32_t bits_in_smem;         // list mode: those two bitmaps are in shared memory
    const long long* lk;          // list mode: every slot's key, largest first, stored as ~key with the top bit flipped
    const int32_t* ls;            //            and the slot it belongs to
    const int64_t* arrival;       // per query: arrival (for the charge pass after the loop)
    struct FastPost* post;        // where list mode began, for the charge pass after the loop
    TreeState* st;
    // trees with a budget: the loop keeps the node arrays of the tree up to date itself (LRU needs them at every decision)
    int32_t lru;                  // 1: the tree has a budget
    int32_t mem_cap;              // entries of the member array (groups formed by evictions are appended behind the first n)
    TreeDev T;
    int32_t* parked;              // per node: unprocessed slots whose hint is that node
    int32_t* hintc;               // per slot: the hint once more, side by side (what the scan after an eviction reads)
    int2* leaf_run;               // per node: the member run that holds every slot whose hint is that node (y < 0: no such run is known)
    long long* pk; int32_t* pi;   // set-up: (hint, slot) pairs, sorted by hint to give every node of the tree its run
    int32_t* skip;                // set by the capacity check before the loop: leave everything untouched
    // a given processing order instead of a policy (klpm_replay): decision c processes query fixed[c]; slots are the
    // queries in index order; *n_fixed decisions are made
    const int32_t* fixed;
    const int32_t* n_fixed;
};

#define KLPM_FAST_THREADS 256
#define KLPM_FAST_SORT_CAP 4096          // largest group that is regrouped exactly (sorted in shared memory)
#define KLPM_FAST_NOGROUP 0xffffffffffffffffULL

__device__ __forceinline__ unsigned long long mix64(unsigned long long z) {      // SplitMix64's finaliser
    z ^= z >> 30; z *= 0xbf58476d1ce4e5b9ULL; z ^= z >> 27; z *= 0x94d049bb133111ebULL; z ^= z >> 31;
    return z;
}
__device__ __forceinline__ unsigned long long group_hash(long long pos, int32_t ntok) {
    return mix64((unsigned long long)(pos + 2) * 0x9E3779B97F4A7C15ULL + (unsigned)ntok) >> 2;
}
__device__ __forceinline__ unsigned long long single_hash(int32_t slot) {       // a query that is fully cached never regroups
    return mix64(0xD1B54A32D192ED03ULL ^ (unsigned long long)(unsigned)slot) >> 2;
}
__device__ __forceinline__ unsigned long long fast_key(int32_t m, int32_t len, int32_t rank, int32_t score_mode) {
    unsigned hi = (unsigned)m;
    if (score_mode == 1) hi = len > 0 ? (unsigned)(((unsigned long long)(unsigned)m << 31) / (unsigned)len) : 0u;
    return ((unsigned long long)hi << 32) | (0xffffffffu - (unsigned)rank);
}
__device__ __forceinline__ FDyn ld_dyn(const FDyn* p) {
    const int4* q = reinterpret_cast<const int4*>(p);
    const int4 a = __ldcg(q), b = __ldcg(q + 1);
    FDyn d;
    d.pos = (long long)(((unsigned long long)(unsigned)a.y << 32) | (unsigned)a.x);
    d.m = a.z; d.ntok = a.w; d.gstart = b.x; d.gcount = b.y; d.hint = b.z; d.pad = 0;
    return d;
}
__device__ __forceinline__ void st_dyn_state(FDyn* p, long long pos, int32_t m, int32_t ntok) {
    __stcg(reinterpret_cast<int4*>(p), make_int4((int)(unsigned)(unsigned long long)pos, (int)(unsigned)((unsigned long long)pos >> 32), m, ntok));
}
__device__ __forceinline__ void st_dyn_group(FDyn* p, int32_t gstart, int32_t gcount) {
    __stcg(reinterpret_cast<int2*>(p) + 2, make_int2(gstart, gcount));
}
__device__ __forceinline__ void st_dyn_hint(FDyn* p, int32_t hint) { __stcg(reinterpret_cast<int32_t*>(p) + 6, hint); }
__device__ __forceinline__ FStat ld_stat(const FStat* p) {
    const int4* q = reinterpret_cast<const int4*>(p);
    const int4 a = __ldg(q), b = __ldg(q + 1);
    FStat s;
    s.t = (long long)(((unsigned long long)(unsigned)a.y << 32) | (unsigned)a.x);
    s.len = a.z; s.ord = a.w;
    s.soff = (long long)(((unsigned long long)(unsigned)b.y << 32) | (unsigned)b.x);
    s.rank = b.z; s.pad = 0;
    return s;
}
__device__ __forceinline__ void named_bar(int id, int nthreads) {
    asm volatile("bar.sync %0, %1;" ::"r"(id), "r"(nthreads) : "memory");
}

// slot -> constant record (after the slots have been ordered by arrival)
__global__ void fast_stat_kernel(const int32_t* __restrict__ ord, const long long* __restrict__ sorted_t,
                                 const int64_t* __restrict__ off, const int32_t* __restrict__ prank, int32_t n, FStat* stat) {
    const int32_t r = blockIdx.x * blockDim.x + threadIdx.x;
    if (r >= n) return;
    const int32_t qi = ord[r];
    const int64_t lo = off[qi];
    FStat s;
    s.soff = lo; s.t = sorted_t[r]; s.len = (int32_t)(off[qi + 1] - lo); s.ord = qi; s.rank = prank ? prank[r] : r; s.pad = 0;
    stat[r] = s;
}

// The hit-rate score is kept as floor(m * 2^31 / |x|) in the high half of a key.  Two different rates m/|x| and
// m'/|x'| differ by at least 1/(|x||x'|), so while every prompt is at most 46,340 tokens long (46,340^2 < 2^31)
// different rates get different quotients, equal rates equal ones, and the order of the keys is the order of the
// rates.  Longer prompts could tie where the rates do not: the status word says so.
#define KLPM_HIT_RATE_MAX_LEN 46340
__global__ void hit_rate_guard_kernel(const int64_t* __restrict__ off, int32_t n, TreeState* st) {
    const int32_t i = blockIdx.x * blockDim.x + threadIdx.x;
    if (i < n && off[i + 1] - off[i] > KLPM_HIT_RATE_MAX_LEN) set_status(st, RT_ERR_INVALID, 109);
}

// Every slot's starting state from the record the batched match wrote for its query (MatchState): match length,
// position, next token; from those its key and the hash of its group.  One thread per slot (and per padding entry
// of the sort that follows).
__global__ void fast_state_kernel(FastArgs A, const MatchState* __restrict__ state, unsigned long long tag, long long np2) {
    const long long r = (long long)blockIdx.x * blockDim.x + threadIdx.x;
    if (r >= np2) return;
    if (r >= A.n) {                                                                        // padding of the sorts
        A.gh[r] = 0x7fffffffffffffffLL; A.gidx[r] = 0x7fffffff;
        if (A.lru) { A.pk[r] = 0x7fffffffffffffffLL; A.pi[r] = 0x7fffffff; }
        return;
    }
    const FStat s = ld_stat(A.stat + r);
    const int4* src = reinterpret_cast<const int4*>(state + s.ord);
    const int4 a = __ldcg(src), b = __ldcg(src + 1);
    const long long pos_in = (long long)(((unsigned long long)(unsigned)a.y << 32) | (unsigned)a.x);
    const long long node_in = (long long)(((unsigned long long)(unsigned)a.w << 32) | (unsigned)a.z);
    int32_t m = b.x, ntok = b.y;
    long long pos = pos_in;
    int32_t hint = 0;
    const unsigned long long got = ((unsigned long long)(unsigned)b.w << 32) | (unsigned)b.z;
    bool bad = got != tag || m < 0 || m > s.len;
    if (A.lru && !bad) { bad = node_in < 0 || node_in >= A.T.max_nodes; hint = (int32_t)node_in; }
    if (bad) {                                       // not the record of that match: say so and start this slot from nothing
        set_status(A.st, RT_ERR_INVALID, 110);
        m = 0; pos = -1; ntok = 0; hint = 0;
    }
    st_dyn_state(A.dyn + r, pos, m, ntok);
    if (A.lru) {
        st_dyn_hint(A.dyn + r, hint); A.hintc[r] = hint; atomicAdd(A.parked + hint, 1);
        A.pk[r] = hint; A.pi[r] = (int32_t)r;
    }
    A.key[r] = fast_key(m, s.len, s.rank, A.score_mode);
    A.gh[r] = (long long)(m < s.len ? group_hash(pos, ntok) : single_hash((int32_t)r));
    A.gidx[r] = (int32_t)r;
}

// Trees with a budget, after the sort by hint: the slots whose match ends in one node, side by side, are that node's
// run (entries n .. 2n-1 of the member array): where the loop looks when the node is evicted with queries parked in it.
__global__ void lru_parklist_kernel(FastArgs A) {
    const int32_t i = blockIdx.x * blockDim.x + threadIdx.x;
    if (i >= A.n) return;
    A.mem[A.n + i] = A.pi[i];
    const long long node = A.pk[i];
    if (i > 0 && A.pk[i - 1] == node) return;              // not the first of its run
    int32_t lo = i + 1, hi = A.n;                          // first index with a larger hint
    while (lo < hi) { const int32_t mid = (lo + hi) >> 1; if (A.pk[mid] <= node) lo = mid + 1; else hi = mid; }
    A.leaf_run[node] = make_int2(A.n + i, lo - i);
}

// after the sort by hash: runs of equal hashes are the groups
__global__ void fast_group_kernel(FastArgs A) {
    const int32_t i = blockIdx.x * blockDim.x + threadIdx.x;
    if (i >= A.n) return;
    const long long h = A.gh[i];
    int32_t lo = 0, hi = i;                    // first index with gh >= h
    while (lo < hi) { const int32_t mid = (lo + hi) >> 1; if (A.gh[mid] < h) lo = mid + 1; else hi = mid; }
    const int32_t first = lo;
    lo = i + 1; hi = A.n;                      // first index with gh > h
    while (lo < hi) { const int32_t mid = (lo + hi) >> 1; if (A.gh[mid] <= h) lo = mid + 1; else hi = mid; }
    const int32_t r = A.gidx[i];
    A.mem[i] = r;
    st_dyn_group(A.dyn + r, first, lo - first);
    if (lo - first > 1) atomicOr(A.gbits + (r >> 5), 1u << (r & 31));
}

// list mode: every slot's key in a form that sorts largest first (padding last)
__global__ void fast_list_kernel(const unsigned long long* __restrict__ key, int32_t n, long long np2, long long* lk, int32_t* ls) {
    const long long i = (long long)blockIdx.x * blockDim.x + threadIdx.x;
    if (i >= np2) return;
    lk[i] = i < n ? (long long)(~key[i] ^ 0x8000000000000000ULL) : 0x7fffffffffffffffLL;
    ls[i] = i < n ? (int32_t)i : 0x7fffffff;
}

// Largest of the warp's 64-bit values with two hardware reductions: the high halves, then the low halves of
// the lanes that hold the largest high half.
__device__ __forceinline__ unsigned long long warp_max64r(unsigned long long v) {
    const unsigned hi = (unsigned)(v >> 32);
    const unsigned mh = __reduce_max_sync(FULL_MASK, hi);
    const unsigned ml = __reduce_max_sync(FULL_MASK, hi == mh ? (unsigned)v : 0u);
    return ((unsigned long long)mh << 32) | ml;
}

// ---- the tournament above the leaf blocks (shared memory) ----
// t1[b] is the largest key of leaf block b among the slots the tournament holds: the arrived, unprocessed slots
// while arrivals are pending; in list mode (everybody has arrived) only those of them whose key has changed since
// the keys were sorted -- the others are picked from the sorted list.
struct FastTour {
    unsigned long long* t1;   // per leaf block (padded with zeros to a multiple of 32)
    unsigned long long* t2;   // per 32 leaf blocks (padded likewise)
    unsigned long long* t3;   // 32 entries
    unsigned int* done;       // bitmap of processed slots (shared memory), or null
    unsigned int* skip;       // bitmap of slots the sorted list must pass over: processed, or key changed (shared memory), or null
    unsigned int* gb;         // bitmap of slots whose group has more than one member (shared memory), or null
    unsigned int* dirty;      // trees with a budget: bitmap of leaf blocks to recompute after a fallback (256 words, shared memory)
    int g_done, g_bits;       // the processed bitmap / the other two bitmaps live in global memory (queues too long for shared memory)
    int32_t n2;               // entries of t2 in use
    int32_t n3;               // entries of t3 in use
};
// A word of one of the loop's bitmaps: shared memory, or global memory read through L2 (other warps set bits with atomics).
__device__ __forceinline__ unsigned bm_ld(const unsigned int* p, long long i, int g) { return g ? __ldcg(p + i) : p[i]; }

// Recompute the ancestors of leaf block b; returns the root.  One warp.
__device__ __forceinline__ unsigned long long tour_update(const FastTour& R, int32_t b, int lane) {
    const int32_t i2 = b >> 5;
    unsigned long long v = warp_max64r(R.t1[(i2 << 5) + lane]);
    if (lane == 0) R.t2[i2] = v;
    __syncwarp();
    const int32_t i3 = i2 >> 5;
    v = warp_max64r(R.t2[(i3 << 5) + lane]);
    if (lane == 0) R.t3[i3] = v;
    __syncwarp();
    return warp_max64r(R.t3[lane]);
}
// Leaf block b's largest key becomes v: write it and its ancestors; returns the root.  One warp; every lane
// performs the same stores, so each lane sees them in its own program order without a barrier.
__device__ __forceinline__ unsigned long long tour_set(const FastTour& R, int32_t b, unsigned long long v, int lane) {
    const int32_t i2 = b >> 5, i3 = i2 >> 5;
    const unsigned long long o1 = warp_max64r(lane == (b & 31) ? 0ULL : R.t1[(i2 << 5) + lane]);
    const unsigned long long o2 = warp_max64r(lane == (i2 & 31) ? 0ULL : R.t2[(i3 << 5) + lane]);
    const unsigned long long o3 = warp_max64r(lane == i3 ? 0ULL : R.t3[lane]);
    const unsigned long long v2 = v > o1 ? v : o1, v3 = v2 > o2 ? v2 : o2;
    R.t1[b] = v; R.t2[i2] = v2; R.t3[i3] = v3;
    return v3 > o3 ? v3 : o3;
}
// Recompute t3 and the root from t2.  One warp.
__device__ __forceinline__ unsigned long long tour_top(const FastTour& R, int lane) {
    for (int32_t i3 = 0; i3 < R.n3; ++i3) {
        const unsigned long long v = warp_max64r(R.t2[(i3 << 5) + lane]);
        if (lane == 0) R.t3[i3] = v;
    }
    __syncwarp();
    return warp_max64r(R.t3[lane]);
}
// Recompute t2 from t1.  Every warp of the CTA; the caller synchronises.
__device__ __forceinline__ void tour_mid(const FastTour& R, int warp, int nwarps, int lane) {
    for (int32_t i2 = warp; i2 < R.n2; i2 += nwarps) {
        const unsigned long long v = warp_max64r(R.t1[(i2 << 5) + lane]);
        if (lane == 0) R.t2[i2] = v;
    }
}
// has slot r been processed?  (the bitmap lives in shared memory when it fits)
__device__ __forceinline__ bool slot_done(const FastTour& R, const FastArgs& A, long long r) {
    const unsigned w = bm_ld(R.done, r >> 5, R.g_done);
    return (w >> (r & 31)) & 1u;
}
// position of the k-th set bit of w (k >= 1, at most the number of set bits)
__device__ __forceinline__ int kth_set_bit(unsigned w, int k) {
    int pos = 0;
    int cnt = __popc(w & 0xffffu); if (k > cnt) { k -= cnt; pos += 16; w >>= 16; }
    cnt = __popc(w & 0xffu);       if (k > cnt) { k -= cnt; pos += 8; w >>= 8; }
    cnt = __popc(w & 0xfu);        if (k > cnt) { k -= cnt; pos += 4; w >>= 4; }
    cnt = __popc(w & 0x3u);        if (k > cnt) { k -= cnt; pos += 2; w >>= 2; }
    if (k > (int)(w & 1u)) pos += 1;
    return pos;
}
__device__ __forceinline__ void set_grouped(const FastTour& R, int32_t r, bool grouped) {
    if (!R.gb) return;
    if (grouped) atomicOr(R.gb + (r >> 5), 1u << (r & 31));
    else atomicAnd(R.gb + (r >> 5), ~(1u << (r & 31)));
}

struct FastPick {             // the prompt being processed, as its group's members need it
    int32_t slot, m, len, ntok;
    const int32_t* x;         // its tokens
    long long pos;
    long long vleaf;          // virtual pool index of the first token of its new leaf
    long long admitted;       // slots below this have arrived
    int32_t gstart, gcount;
    int32_t leaf;             // trees with a budget: id of its new leaf (the tied members are parked in it from now on)
};
struct FastJob { int32_t type; int32_t a0, a1; FastPick pick; };
enum { FAST_JOB_EXIT = 0, FAST_JOB_ADMIT = 1, FAST_JOB_DISSOLVE = 2, FAST_JOB_REBUILD = 3, FAST_JOB_BATCH = 4, FAST_JOB_FALLBACK = 5 };

// trees with a budget: slot r's match now ends inside node `to` (it was counted for node `from`)
__device__ __forceinline__ void lru_move(const FastArgs& A, int32_t r, int32_t from, int32_t to) {
    st_dyn_hint(A.dyn + r, to);
    __stcg(A.hintc + r, to);
    atomicSub(A.parked + from, 1);
    atomicAdd(A.parked + to, 1);
}

// List mode: the largest key among the unprocessed slots of leaf block b whose key has changed since the sort.  One warp.
__device__ __forceinline__ unsigned long long changed_block_max(const FastArgs& A, const FastTour& R, int32_t b, int lane) {
    unsigned long long v = 0;
    for (int32_t u = lane; u < (1 << A.lb_shift); u += 32) {
        const long long r = ((long long)b << A.lb_shift) + u;
        if (r < A.n) {
            const unsigned w = bm_ld(R.skip, r >> 5, R.g_bits) & ~bm_ld(R.done, r >> 5, R.g_done);
            if ((w >> (r & 31)) & 1u) { const unsigned long long kk = __ldcg(A.key + r); if (kk > v) v = kk; }
        }
    }
    return warp_max64r(v);
}

// What the sequencer hands to a CTA-wide batch of decisions, and what it gets back.
struct FastBatchIO {
    int32_t cur, head, c, cyc;        // in: list cursor, oldest unprocessed slot, decisions made, c mod k
    unsigned long long root;          // in: largest key in the tournament
    int32_t B, consumed, hmax;        // out: decisions made (0: none), list entries passed, last slot taken by an oldest-first turn
    int32_t B0, Bmax, limF, limL;     // scratch
    // scratch: the slots both kinds of turn reach inside the batch (rank among the oldest-first picks, rank among the
    // list entries), and after they are resolved the ranks each side passes over, ascending
    int32_t ncol, nRH, nRE;
    int32_t colPhi[32], colRk[32], remH[32], remE[32];
    int32_t hard;                     // out: the batch stopped before a decision that needs the one-at-a-time path
    int32_t Braw;                     // out: decisions the batch could have made (it makes none below KLPM_FAST_CTA_MIN)
    int32_t limB;                     // scratch: the batch must end before this decision (list entries that an oldest-first pick would meet)
};
#define KLPM_FAST_CTA_BATCH 1024      // decisions per CTA-wide batch at most (4 list entries per thread)
#ifndef KLPM_FAST_CTA_MIN
#define KLPM_FAST_CTA_MIN 32         // smaller batches are left to the warp-wide step (an attempt costs about 10,000 cycles)
#endif
#ifndef KLPM_FAST_CB_MAX
#define KLPM_FAST_CB_MAX 32           // longest back-off (loop iterations) after CTA-wide attempts that failed
#endif
#ifndef KLPM_FAST_FAIL_CAP
#define KLPM_FAST_FAIL_CAP 6          // failed CTA-wide attempts in a row that still lengthen the wait (8 << that many decisions)
#endif
#ifndef KLPM_FAST_CALM
#define KLPM_FAST_CALM 1              // full warp-wide steps in a row before a CTA-wide batch is tried again
#endif

// Exclusive prefix sum of v over the CTA's 256 threads; *total receives the sum.  s_w: 8 ints of shared scratch.
__device__ __forceinline__ int32_t block_excl_scan(int32_t v, int32_t* s_w, int32_t* total) {
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    int32_t inc = v;
#pragma unroll
    for (int d = 1; d < 32; d <<= 1) { const int32_t o = __shfl_up_sync(FULL_MASK, inc, d); if (lane >= d) inc += o; }
    __syncthreads();                   // s_w may still be read from an earlier scan
    if (lane == 31) s_w[warp] = inc;
    __syncthreads();
    int32_t before = 0, all = 0;
#pragma unroll
    for (int w = 0; w < KLPM_FAST_THREADS / 32; ++w) { const int32_t x = s_w[w]; if (w < warp) before += x; all += x; }
    *total = all;
    return before + inc - v;
}

// One member of the dissolving group per lane (r < 0: none).  Members tied with the processed prompt are
// compared with its uncached tokens and get their new state and key; every live member gets the hash of the
// group it belongs to from now on (KLPM_FAST_NOGROUP: it leaves the run).  *touched: its key grew and it
// has arrived, so its leaf block's ancestors need recomputing.  Warp-cooperative.
__device__ __forceinline__ unsigned long long fast_member(const FastArgs& A, const FastPick& P, const FastTour& R, int32_t r, int lane,
                                                          bool* touched) {
    const bool act = r >= 0 && r != P.slot;
    FDyn d; d.pos = 0; d.m = -1; d.ntok = 0; d.gstart = 0; d.gcount = 0;
    FStat s; s.soff = 0; s.t = 0; s.len = 0; s.ord = 0; s.rank = 0;
    if (act) { d = ld_dyn(A.dyn + r); s = ld_stat(A.stat + r); }
    const bool live = act && !slot_done(R, A, r);
    const bool tied = live && d.pos == P.pos && d.ntok == P.ntok && d.m == P.m && d.m < s.len;
    const int32_t* q = A.tok + s.soff;
    int32_t e = 0;
    unsigned cm = __ballot_sync(FULL_MASK, tied);
    while (cm) {
        const int src = __ffs(cm) - 1; cm &= cm - 1;
        const int32_t* qq = (const int32_t*)__shfl_sync(FULL_MASK, (unsigned long long)q, src);
        const int32_t ql = __shfl_sync(FULL_MASK, s.len, src);
        const int32_t lim = (ql < P.len ? ql : P.len) - P.m;
        const int32_t ee = first_mismatch<true>(qq + P.m, P.x + P.m, lim);
        if (lane == src) e = ee;
    }
    *touched = false;
    if (tied) {
        d.m = P.m + e; d.pos = P.vleaf + e - 1; d.ntok = d.m < s.len ? __ldg(q + d.m) : 0;
        st_dyn_state(A.dyn + r, d.pos, d.m, d.ntok);
        if (A.lru) lru_move(A, r, d.hint, P.leaf);
        const unsigned long long key = fast_key(d.m, s.len, s.rank, A.score_mode);
        __stcg(A.key + r, key);
        if (R.skip) atomicOr(R.skip + (r >> 5), 1u << (r & 31));          // its entry of the sorted list is stale now
        if ((long long)r < P.admitted) { atomicMax(R.t1 + (r >> A.lb_shift), key); *touched = true; }
    }
    if (!live) return KLPM_FAST_NOGROUP;
    return d.m < s.len ? group_hash(d.pos, d.ntok) : single_hash(r);
}

// The warp-wide step of list mode (see fast_run_kernel) with the whole CTA: 1,024 list entries and 8,192 bitmap slots
// are examined at once, the same checks cut the batch short, block-wide prefix sums replace the warp's ballots.
// Every thread calls it.  Nothing is changed unless at least KLPM_FAST_CTA_MIN decisions can be made.
template <bool G>
__device__ void fast_batch_job(const FastArgs& A, const FastTour& R0, FastBatchIO* io, int32_t* sH, int32_t* sE, int32_t* sEpos,
                               int32_t* sF, int32_t* s_w, int32_t nwords) {
    FastTour R = R0;                                        // with the bitmaps in shared memory the flags fold away
    if (!G) { R.g_done = 0; R.g_bits = 0; }
    const int tid = threadIdx.x;
    const int32_t n = A.n, cur = io->cur, head = io->head, c = io->c, cyc = io->cyc;
    const unsigned long long root = io->root;
    // the list entries cur + 4 tid .. + 3 (asked for first: the table below is filled while they travel)
    long long kk[4]; int32_t es[4]; bool ok[4];
#pragma unroll
    for (int r = 0; r < 4; ++r) {
        const long long idx = (long long)cur + tid * 4 + r;
        kk[r] = 0; es[r] = 0;
        if (idx < n) { kk[r] = __ldg(A.lk + idx); es[r] = __ldg(A.ls + idx); }
    }
    // sF[x] = oldest-first turns among the next x decisions, x = 0 .. 1,024.  Under k-LPM the first such turn is
    // decision (k - cyc) mod k and then every k-th, which is floor((x + s) / k) with s = (cyc + k - 1) mod k; one
    // division per thread, the later entries follow by adding 256 = Q k + Rm.
    {
        const int32_t sft = cyc == 0 ? A.k - 1 : cyc - 1;
        int32_t q = 0, rem = 0, Q = 0, Rm = 0;
        if (A.policy == KLPM_POLICY_KLPM) { q = (tid + sft) / A.k; rem = (tid + sft) - q * A.k; Q = KLPM_FAST_THREADS / A.k; Rm = KLPM_FAST_THREADS - Q * A.k; }
        for (int32_t x = tid; x <= KLPM_FAST_CTA_BATCH; x += KLPM_FAST_THREADS) {
            sF[x] = A.policy == KLPM_POLICY_FCFS ? x : A.policy == KLPM_POLICY_LPM ? 0 : q;
            q += Q; rem += Rm;
            if (rem >= A.k) { rem -= A.k; ++q; }
        }
    }
    // the limits start open; every thread reads them capped by what the batch can hold
    if (tid == 0) { io->B0 = 0; io->Bmax = 0; io->limF = 0x7fffffff; io->limL = 0x7fffffff; io->limB = 0x7fffffff; io->ncol = 0; io->nRH = 0; io->nRE = 0; }
    auto f = [&](int32_t x) -> int32_t { return sF[x]; };
    // those of the entries that still count
    int32_t cnt = 0;
#pragma unroll
    for (int r = 0; r < 4; ++r) {
        const long long idx = (long long)cur + tid * 4 + r;
        ok[r] = idx < n && !((bm_ld(R.skip, es[r] >> 5, R.g_bits) >> (es[r] & 31)) & 1u);
        cnt += ok[r];
    }
    // the unprocessed slots from `head` on, one bitmap word per thread
    const int32_t w0 = head >> 5;
    unsigned fr;
    {
        const int32_t wi = w0 + tid;
        unsigned w = wi < nwords ? bm_ld(R.done, wi, R.g_done) : 0xffffffffu;
        if (wi == nwords - 1 && (n & 31)) w |= ~((1u << (n & 31)) - 1u);
        if (wi == w0) w |= (1u << (head & 31)) - 1u;
        fr = ~w;
    }
    // both prefix sums with one scan: usable entries (at most 1,024) in the low half, free slots (at most 8,192) above
    int32_t both;
    const int32_t base2 = block_excl_scan(cnt + (__popc(fr) << 16), s_w, &both);    // (its barriers also publish sF and the limits)
    const int32_t base = base2 & 0xffff, qk = base2 >> 16;
    const int32_t avail = both & 0xffff, nfree = both >> 16;
    int32_t* sP = sF + KLPM_FAST_CTA_BATCH + 8;             // per word: free slots before it
    unsigned* sFr = reinterpret_cast<unsigned*>(sP + KLPM_FAST_THREADS);
    sP[tid] = qk; sFr[tid] = fr;
    {   // as many decisions as those entries allow: the largest x with x - f(x) <= avail, every thread trying four values
        const int32_t hi = n - c < KLPM_FAST_CTA_BATCH ? n - c : KLPM_FAST_CTA_BATCH;
        int32_t best = 0;
#pragma unroll
        for (int r = 1; r <= 4; ++r) { const int32_t x = tid * 4 + r; if (x <= hi && x - f(x) <= avail) best = x; }
        best = __reduce_max_sync(FULL_MASK, best);
        if ((tid & 31) == 0 && best > 0) atomicMax(&io->B0, best);
    }
    __syncthreads();
    const int32_t B0 = io->B0, nF0 = f(B0), nL0 = B0 - nF0;
    // One slot and one entry more than a full batch takes are looked at: where the two pick orders meet once inside the
    // batch (a slot that is both among the oldest unprocessed and among the next list entries), the side that comes
    // later passes over it and takes one more of its own.
    const bool both_kinds = A.policy == KLPM_POLICY_KLPM && A.k >= 2;       // (k = 1: every turn is an oldest-first turn)
    const int32_t nFw = both_kinds ? (nF0 + 32 < KLPM_FAST_CTA_BATCH ? nF0 + 32 : KLPM_FAST_CTA_BATCH) : nF0;
    const int32_t nLw = both_kinds ? (nL0 + 32 < KLPM_FAST_CTA_BATCH ? nL0 + 32 : KLPM_FAST_CTA_BATCH) : nL0;
    const int32_t nFa = nfree < nFw ? nfree : nFw;          // oldest-first picks there are slots for
    const int32_t nEa = avail < nLw ? avail : nLw;          // longest-match picks there are entries for
    // the next nFa unprocessed slots in order: a thread per slot, eight words at a time; the slot's rank among the free
    // ones is where it goes; one whose key sits in the tournament or that is grouped needs the careful step
    {
        const int bit = tid & 31;
        for (int32_t wl = tid >> 5; wl < KLPM_FAST_THREADS && sP[wl] < nFa; wl += KLPM_FAST_THREADS / 32) {
            const unsigned fw = sFr[wl];
            if ((fw >> bit) & 1u) {
                const int32_t rank = sP[wl] + __popc(fw & ((1u << bit) - 1u));
                if (rank < nFa) {
                    const int32_t hs = (w0 + wl) * 32 + bit;
                    sH[rank] = hs;
                    if (((bm_ld(R.skip, hs >> 5, R.g_bits) | bm_ld(R.gb, hs >> 5, R.g_bits)) >> (hs & 31)) & 1u) atomicMin(&io->limF, rank);
                }
            }
        }
    }
    __syncthreads();
    const int32_t hmax0 = nFa > 0 ? sH[nFa - 1] : -1;
    // The usable entries by rank.  One that is grouped or lies below the tournament's root stops the batch before its
    // turn.  One whose slot is among the slots the oldest-first picks would take (rank phi there) is taken by whichever
    // side reaches it first.  The first such meeting (the one whose earlier decision comes first) is resolved inside
    // the batch: the other side passes over the slot, its later picks move up by one.  The batch ends well before any
    // further meeting: k + 1 decisions before the earlier of its two decisions as computed without the shift, which
    // moves a decision forward by at most k -- or before the later of its two decisions where those are far enough
    // apart for the shift not to change their order (the earlier one is an ordinary pick then).
    {
        int32_t rk = base;
#pragma unroll
        for (int r = 0; r < 4; ++r) {
            if (ok[r]) {
                if (rk < nEa) {
                    sE[rk] = es[r]; sEpos[rk] = tid * 4 + r;
                    const unsigned long long ek = ~((unsigned long long)kk[r] ^ 0x8000000000000000ULL);
                    if ((((bm_ld(R.gb, es[r] >> 5, R.g_bits) >> (es[r] & 31)) & 1u)) || root > ek) {
                        atomicMin(&io->limL, rk);
                    } else if (es[r] >= head && es[r] <= hmax0) {
                        int32_t lo = 0, hi = nFa;                        // phi: slots of sH before this one
                        while (lo < hi) { const int32_t mid = (lo + hi) >> 1; if (sH[mid] < es[r]) lo = mid + 1; else hi = mid; }
                        const int32_t phi = lo;
                        // decision of the oldest-first turn of rank phi, and of the longest-match turn of rank rk
                        int32_t xF, xL;
                        if (A.policy == KLPM_POLICY_FCFS) { xF = phi; xL = B0; }
                        else if (A.policy == KLPM_POLICY_LPM) { xF = B0; xL = rk; }
                        else {
                            const int32_t i0 = cyc == 0 ? 0 : A.k - cyc;
                            const long long xF64 = i0 + (long long)phi * A.k;
                            xF = xF64 < 0x3ffffff ? (int32_t)xF64 : 0x3ffffff;
                            xL = rk;                                       // before the first oldest-first turn; after it k - 1 of every k decisions
                            if (rk >= i0 && A.k >= 2) {
                                const int32_t u1 = rk - i0, q = u1 / (A.k - 1);
                                const long long xL64 = i0 + (long long)q * A.k + 1 + (u1 - q * (A.k - 1));
                                xL = xL64 < 0x3ffffff ? (int32_t)xL64 : 0x3ffffff;
                            }
                        }
                        // without resolving: the batch would have to end before the later of the two decisions (used
                        // when there are more such slots than the resolution below takes)
                        atomicMin(&io->limB, xF > xL ? xF : xL);
                        if (both_kinds) {
                            const int32_t ci = atomicAdd(&io->ncol, 1);
                            if (ci < 32) { io->colPhi[ci] = phi; io->colRk[ci] = rk; }
                        }
                    }
                }
                ++rk;
            }
        }
    }
    __syncthreads();
    // Where the two orders meet, sequential processing gives the slot to whichever turn comes first, and the other side
    // passes over it: its later picks move up by one.  Warp 0 plays the meetings through in the order of their first
    // decision (lane i holds meeting i; the time at which a side reaches a slot is its rank minus the ranks below it
    // that this side has passed over so far, turned into a decision number; the earliest pending decision is final,
    // because whatever happens later moves later picks only).  Result: the ranks each side passes over, ascending.
    const int32_t ncol = io->ncol;                          // (block-uniform)
    const bool resolve = both_kinds && ncol > 0 && ncol <= 32;
    if (resolve) {
        if (tid < 32) {
            const int lane = tid;
            const bool mine = lane < ncol;
            const int32_t phi = mine ? io->colPhi[lane] : 0x7fffffff, rk = mine ? io->colRk[lane] : 0x7fffffff;
            unsigned belowPhi = 0, belowRk = 0;             // meetings with a smaller rank on either side
            for (int j = 0; j < ncol; ++j) {
                const int32_t pj = __shfl_sync(FULL_MASK, phi, j), rj = __shfl_sync(FULL_MASK, rk, j);
                if (pj < phi) belowPhi |= 1u << j;
                if (rj < rk) belowRk |= 1u << j;
            }
            const int32_t i0 = cyc == 0 ? 0 : A.k - cyc;    // decisions before the first oldest-first turn
            const long long FAR = 0x3ffffff;
            // decision of the longest-match turn of rank u, of the oldest-first turn of rank t
            auto l_turn = [&](int32_t u) -> long long {
                if (u < i0) return u;
                const int32_t u1 = u - i0, q = u1 / (A.k - 1);
                return i0 + (long long)q * A.k + 1 + (u1 - q * (A.k - 1));
            };
            // no batch gets past the first slot or entry that needs the careful step, whoever passes over what
            const int32_t capF = io->limF < nFa ? io->limF : nFa, capL = io->limL < nEa ? io->limL : nEa;
            long long bcap = B0;
            { const long long a1 = i0 + (long long)capF * A.k, a2 = l_turn(capL); if (a1 < bcap) bcap = a1; if (a2 < bcap) bcap = a2; }
            long long xF = FAR, xL = FAR;
            if (mine) { xF = i0 + (long long)phi * A.k; xL = l_turn(rk); if (xF > FAR) xF = FAR; }
            unsigned remH = 0, remE = 0, open_ = ncol == 32 ? 0xffffffffu : ((1u << ncol) - 1u);
            while (open_) {
                unsigned key = 0xffffffffu;
                const bool l_first = xL < xF;
                if (mine && ((open_ >> lane) & 1u)) key = ((unsigned)(l_first ? xL : xF) << 5) | (unsigned)lane;
                const unsigned win = __reduce_min_sync(FULL_MASK, key);
                if ((long long)(win >> 5) >= bcap) break;   // beyond what the batch can reach: nothing more to settle
                const int wl = (int)(win & 31u);
                const bool wl_first = __shfl_sync(FULL_MASK, (int)l_first, wl) != 0;
                open_ &= ~(1u << wl);
                if (wl_first) {                             // a longest-match turn took that slot: later oldest-first picks come one turn earlier
                    remH |= 1u << wl;
                    if (((belowPhi >> wl) & 1u) && xF < FAR) xF -= A.k;
                } else {                                    // an oldest-first turn took that entry's slot: later list picks come one turn earlier
                    remE |= 1u << wl;
                    if ((belowRk >> wl) & 1u) {
                        long long y = xL - 1;
                        if (y >= i0 && (y - i0) % A.k == 0) --y;       // (that one is an oldest-first turn)
                        xL = y;
                    }
                }
            }
            if (mine && ((remH >> lane) & 1u)) io->remH[__popc(remH & belowPhi)] = phi;
            if (mine && ((remE >> lane) & 1u)) io->remE[__popc(remE & belowRk)] = rk;
            if (lane == 0) { io->nRH = __popc(remH); io->nRE = __popc(remE); }
        }
        __syncthreads();
    }
    // the limits, capped by what is in sight
    const int32_t limF = io->limF < nFa ? io->limF : nFa, limL = io->limL < nEa ? io->limL : nEa;
    const int32_t limB = resolve || io->limB > B0 ? B0 : io->limB;
    const int32_t nRH = io->nRH, nRE = io->nRE;
    // rank t among the oldest-first picks -> index of its slot in sH; rank u among the longest-match picks -> index in sE
    auto hI = [&](int32_t t) -> int32_t { for (int32_t j = 0; j < nRH; ++j) { if (io->remH[j] <= t) ++t; else break; } return t; };
    auto eI = [&](int32_t u) -> int32_t { for (int32_t j = 0; j < nRE; ++j) { if (io->remE[j] <= u) ++u; else break; } return u; };
    {   // the largest x that respects the limits, every thread trying four values
        int32_t best = 0;
#pragma unroll
        for (int r = 1; r <= 4; ++r) {
            const int32_t x = tid * 4 + r, nf = f(x), nl = x - nf;
            if (x <= limB && (nf == 0 || hI(nf - 1) < limF) && (nl == 0 || eI(nl - 1) < limL)) best = x;
        }
        best = __reduce_max_sync(FULL_MASK, best);
        if ((tid & 31) == 0 && best > 0) atomicMax(&io->Bmax, best);
    }
    __syncthreads();
    const int32_t Braw = io->Bmax;
    const int32_t B = Braw >= KLPM_FAST_CTA_MIN ? Braw : 0;     // nothing is changed by a batch too short to pay
    if (tid == 0) {
        const int32_t nF = f(B), nL = B - nF;
        io->B = B; io->Braw = Braw;
        io->consumed = nL > 0 ? sEpos[eI(nL - 1)] + 1 : 0;
        io->hmax = nF > 0 ? sH[hI(nF - 1)] : -1;
        // stopped by a decision only the one-at-a-time path can take (not by the end of what is in sight, nor by a
        // further slot both kinds of turn reach: the next batch sorts that out)
        const int32_t nf1 = f(B + 1), nl1 = B + 1 - nf1;
        io->hard = B > 0 && B < B0 && ((nf1 > 0 && hI(nf1 - 1) >= io->limF) || (nl1 > 0 && eI(nl1 - 1) >= io->limL)) ? 1 : 0;
    }
    for (int32_t x = tid; x < B; x += KLPM_FAST_THREADS) {   // thread makes decisions c + x
        const int32_t f0 = f(x);
        const int32_t slot = f(x + 1) > f0 ? sH[hI(f0)] : sE[eI(x - f0)];
        atomicOr(R.done + (slot >> 5), 1u << (slot & 31));
        atomicOr(R.skip + (slot >> 5), 1u << (slot & 31));
        A.order[c + x] = slot;
    }
    __syncthreads();
}

// sh[0..p2) / sr[0..p2) hold the group hash and the slot of cnt members (padded with KLPM_FAST_NOGROUP / -1 up to the
// power of two p2): sort them by hash and write them to the member array from `gs` on, every member with the run of
// equal hashes it is in as its group.  Every thread of the CTA calls it.
__device__ void sort_and_group(const FastArgs& A, const FastTour& R, unsigned long long* sh, int32_t* sr, int32_t cnt, int32_t p2, int32_t gs) {
    const int tid = threadIdx.x, nthr = blockDim.x;
    for (int32_t k = 2; k <= p2; k <<= 1)
        for (int32_t j = k >> 1; j > 0; j >>= 1) {
            for (int32_t i = tid; i < p2; i += nthr) {
                const int32_t l = i ^ j;
                if (l > i) {
                    const unsigned long long a = sh[i], b = sh[l];
                    if ((a > b) == ((i & k) == 0)) { sh[i] = b; sh[l] = a; const int32_t t = sr[i]; sr[i] = sr[l]; sr[l] = t; }
                }
            }
            __syncthreads();
        }
    for (int32_t i = tid; i < cnt; i += nthr) {
        const unsigned long long h = sh[i];
        if (h == KLPM_FAST_NOGROUP) continue;
        int32_t lo = 0, hi = i;
        while (lo < hi) { const int32_t mid = (lo + hi) >> 1; if (sh[mid] < h) lo = mid + 1; else hi = mid; }
        const int32_t first = lo;
        lo = i + 1; hi = cnt;
        while (lo < hi) { const int32_t mid = (lo + hi) >> 1; if (sh[mid] <= h) lo = mid + 1; else hi = mid; }
        const int32_t r = sr[i];
        __stcg(A.mem + gs + i, r);
        st_dyn_group(A.dyn + r, gs + first, lo - first);
        set_grouped(R, r, lo - first > 1);
    }
}

// The same for more members than the shared-memory scratch holds: A.gh[0..cnt) / A.gidx[0..cnt) hold hash and slot.  A
// bitonic sort of the arrays in global memory -- partner distances of a tile (4,096) and more one pass over global
// memory each, everything below inside shared memory tile by tile -- then the runs of equal hashes become the groups.
__device__ void sort_large_and_group(const FastArgs& A, const FastTour& R, unsigned long long* sh, int32_t* sr, int32_t cnt, int32_t gs) {
    const int tid = threadIdx.x, nthr = blockDim.x;
    constexpr int32_t TILE = KLPM_FAST_SORT_CAP;
    int32_t p2 = TILE;
    while (p2 < cnt) p2 <<= 1;
    for (int32_t i = cnt + tid; i < p2; i += nthr) { __stcg(A.gh + i, (long long)KLPM_FAST_NOGROUP); __stcg(A.gidx + i, -1); }
    __syncthreads();
    // stages k_lo .. k_hi (or the tail of one stage) on every tile, in shared memory
    auto tiles = [&](int32_t k_lo, int32_t k_hi) {
        for (int32_t base = 0; base < p2; base += TILE) {
            for (int32_t i = tid; i < TILE; i += nthr) { sh[i] = (unsigned long long)__ldcg(A.gh + base + i); sr[i] = __ldcg(A.gidx + base + i); }
            __syncthreads();
            for (int32_t k = k_lo; k <= k_hi; k <<= 1) {
                const int32_t jmax = (k >> 1) < (TILE >> 1) ? (k >> 1) : (TILE >> 1);
                for (int32_t j = jmax; j > 0; j >>= 1) {
                    for (int32_t i = tid; i < TILE; i += nthr) {
                        const int32_t l = i ^ j;
                        if (l > i) {
                            const unsigned long long a = sh[i], b = sh[l];
                            if ((a > b) == (((base + i) & k) == 0)) { sh[i] = b; sh[l] = a; const int32_t t = sr[i]; sr[i] = sr[l]; sr[l] = t; }
                        }
                    }
                    __syncthreads();
                }
            }
            for (int32_t i = tid; i < TILE; i += nthr) { __stcg(A.gh + base + i, (long long)sh[i]); __stcg(A.gidx + base + i, sr[i]); }
            __syncthreads();
        }
    };
    tiles(2, TILE);
    for (int32_t k = TILE << 1; k <= p2; k <<= 1) {
        for (int32_t j = k >> 1; j >= TILE; j >>= 1) {
            for (int32_t i = tid; i < p2; i += nthr) {
                const int32_t l = i ^ j;
                if (l > i) {
                    const unsigned long long a = (unsigned long long)__ldcg(A.gh + i), b = (unsigned long long)__ldcg(A.gh + l);
                    if ((a > b) == ((i & k) == 0)) {
                        const int32_t ri = __ldcg(A.gidx + i), rl = __ldcg(A.gidx + l);
                        __stcg(A.gh + i, (long long)b); __stcg(A.gh + l, (long long)a); __stcg(A.gidx + i, rl); __stcg(A.gidx + l, ri);
                    }
                }
            }
            __syncthreads();
        }
        tiles(k, k);
    }
    // runs of equal hashes; nearly every member is alone, which its two neighbours show
    for (int32_t i = tid; i < cnt; i += nthr) {
        const unsigned long long h = (unsigned long long)__ldcg(A.gh + i);
        if (h == KLPM_FAST_NOGROUP) continue;
        int32_t first = i, last = i + 1;
        if (i > 0 && (unsigned long long)__ldcg(A.gh + i - 1) == h) {
            int32_t lo = 0, hi = i;
            while (lo < hi) { const int32_t mid = (lo + hi) >> 1; if ((unsigned long long)__ldcg(A.gh + mid) < h) lo = mid + 1; else hi = mid; }
            first = lo;
        }
        if (i + 1 < cnt && (unsigned long long)__ldcg(A.gh + i + 1) == h) {
            int32_t lo = i + 1, hi = cnt;
            while (lo < hi) { const int32_t mid = (lo + hi) >> 1; if ((unsigned long long)__ldcg(A.gh + mid) <= h) lo = mid + 1; else hi = mid; }
            last = lo;
        }
        const int32_t r = __ldcg(A.gidx + i);
        __stcg(A.mem + gs + i, r);
        st_dyn_group(A.dyn + r, gs + first, last - first);
        set_grouped(R, r, last - first > 1);
    }
}

// t1 of leaf block b: the largest key among its arrived (< a1), unprocessed slots.  One warp.
__device__ __forceinline__ void admit_blocks_one(const FastArgs& A, const FastTour& R, int32_t b, int32_t lo_slot, int32_t a1, int lane) {
    unsigned long long v = 0;
    for (int32_t u = lane; u < (1 << A.lb_shift); u += 32) {
        const long long r = (long long)lo_slot + u;
        if (r < a1 && !slot_done(R, A, r)) { const unsigned long long kk = __ldcg(A.key + r); if (kk > v) v = kk; }
    }
    v = warp_max64r(v);
    if (lane == 0) R.t1[b] = v;
}

// t1 of every leaf block that holds a slot of [a0, a1): the largest key among its arrived (< a1), unprocessed slots.
__device__ void admit_blocks(const FastArgs& A, const FastTour& R, int32_t a0, int32_t a1) {
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5, nwarps = blockDim.x >> 5;
    if (a1 <= a0) return;
    const int32_t b0 = a0 >> A.lb_shift, b1 = (a1 - 1) >> A.lb_shift;
    const int32_t LB = 1 << A.lb_shift;
    for (int32_t b = b0 + warp; b <= b1; b += nwarps) {
        unsigned long long v = 0;
        for (int32_t u = lane; u < LB; u += 32) {
            const long long r = ((long long)b << A.lb_shift) + u;
            if (r < a1 && !slot_done(R, A, r)) { const unsigned long long kk = __ldcg(A.key + r); if (kk > v) v = kk; }
        }
        v = warp_max64r(v);
        if (lane == 0) R.t1[b] = v;
    }
}

// Work the whole CTA shares; every thread calls it with the same job.  Ends with t2 recomputed from t1.
__device__ void fast_job(const FastArgs& A, const FastTour& R, const FastJob& J, unsigned long long* sh, int32_t* sr, int* s_cnt,
                         int32_t* s_memcur) {
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5, nwarps = blockDim.x >> 5;
    const int tid = threadIdx.x, nthr = blockDim.x;
    if (J.type == FAST_JOB_ADMIT) {
        // slots [a0, a1) have arrived: the largest key of every leaf block they fall into
        admit_blocks(A, R, J.a0, J.a1);
    } else if (J.type == FAST_JOB_FALLBACK) {
        // Trees with a budget: a leaf in which queries were parked has been evicted.  Every unprocessed slot whose hint
        // is a dead node walks up to the node its match ends in now; the slots that lose matched tokens that way (the
        // match ended inside an evicted leaf) end at the end of a live node's edge, get their new state and key, and
        // are grouped afresh in a run appended to the member array: everybody who falls back to one position with one
        // next token is in this batch (a query parked there before would have matched into the leaf that was there).
        if (tid == 0) *s_cnt = 0;
        for (int32_t i = tid; i < 256; i += nthr) R.dirty[i] = 0u;
        __syncthreads();
        // slots below a0 (the oldest unprocessed slot) are all processed; four hints, then four dead flags, in flight per thread
        for (int32_t r0 = J.a0 + tid; r0 < A.n; r0 += 4 * nthr) {
            int32_t hh[4];
            bool dd[4];
#pragma unroll
            for (int u = 0; u < 4; ++u) { const int32_t r = r0 + u * nthr; hh[u] = r < A.n ? __ldcg(A.hintc + r) : 0; }
#pragma unroll
            for (int u = 0; u < 4; ++u) dd[u] = hh[u] != 0 && __ldcg(A.T.dead + hh[u]) != 0;
#pragma unroll
            for (int u = 0; u < 4; ++u) {
                const int32_t r = r0 + u * nthr, h = hh[u];
                if (!dd[u] || slot_done(R, A, r)) continue;
                const int32_t* dp = reinterpret_cast<const int32_t*>(A.dyn + r);
                const int32_t m0 = __ldcg(dp + 2);
                int32_t m = m0, a = h;
                while (a != 0) {
                    const bool dead = __ldcg(A.T.dead + a) != 0;
                    const int32_t ds = __ldcg(A.T.depth_start + a);
                    if (dead) { if (ds < m) m = ds; }
                    else if (m > ds) break;
                    a = __ldcg(A.T.parent + a);
                }
                st_dyn_hint(A.dyn + r, a);
                __stcg(A.hintc + r, a);
                atomicAdd(A.parked + a, 1);                  // (what the dead node was counted for no longer matters)
                A.leaf_run[a].y = -1;                        // slots from elsewhere are parked in a now: no one run holds them all
                if (m != m0) {
                    const FStat s = ld_stat(A.stat + r);
                    const long long pos = a == 0 ? -1 : __ldcg(A.T.span_off + a) + (long long)(m - __ldcg(A.T.depth_start + a)) - 1;
                    const int32_t ntok = __ldg(A.tok + s.soff + m);                 // m < m0 <= length
                    st_dyn_state(A.dyn + r, pos, m, ntok);
                    __stcg(A.key + r, fast_key(m, s.len, s.rank, A.score_mode));
                    if (r < J.a1) { const int32_t b = r >> A.lb_shift; atomicOr(R.dirty + (b >> 5), 1u << (b & 31)); }
                    const int32_t k = atomicAdd(s_cnt, 1);
                    __stcg(A.gh + k, (long long)group_hash(pos, ntok));
                    __stcg(A.gidx + k, r);
                }
            }
        }
        __syncthreads();
        const int32_t F = *s_cnt, base = *s_memcur;
        __syncthreads();
        if (F > 0) {
            if ((long long)base + F > (long long)A.mem_cap) {
                if (tid == 0) set_status(A.st, RT_ERR_CAPACITY, 113);      // no room for the new groups: the results are void
            } else {
                if (tid == 0) *s_memcur = base + F;
                if (F <= KLPM_FAST_SORT_CAP) {
                    int32_t p2 = 1;
                    while (p2 < F) p2 <<= 1;
                    for (int32_t i = tid; i < p2; i += nthr) {
                        sh[i] = i < F ? (unsigned long long)__ldcg(A.gh + i) : KLPM_FAST_NOGROUP;
                        sr[i] = i < F ? __ldcg(A.gidx + i) : -1;
                    }
                    __syncthreads();
                    sort_and_group(A, R, sh, sr, F, p2, base);
                } else {
                    sort_large_and_group(A, R, sh, sr, F, base);
                }
            }
        }
        __syncthreads();
        // keys went down: the leaf blocks that hold an arrived slot which fell back are recomputed
        for (int32_t w = warp; w < 256; w += nwarps) {
            unsigned bits = R.dirty[w];
            while (bits) {
                const int32_t b = w * 32 + __ffs(bits) - 1;
                bits &= bits - 1;
                const int32_t lo_slot = b << A.lb_shift;
                admit_blocks_one(A, R, b, lo_slot, J.a1, lane);
            }
        }
    } else if (J.type == FAST_JOB_REBUILD) {
        // entering list mode (32-slot leaf blocks): the tournament keeps only the unprocessed slots whose key has changed
        for (int32_t b = warp; b < A.nb; b += nwarps) {
            const unsigned long long v = changed_block_max(A, R, b, lane);
            if (lane == 0) R.t1[b] = v;
        }
    } else {
        // dissolve a group of more than 32 members, or a smaller one whose members have long compares ahead
        const FastPick& P = J.pick;
        const int32_t gs = P.gstart, gc = P.gcount;
        const bool exact = gc <= KLPM_FAST_SORT_CAP;
        int32_t p2 = 1;
        while (p2 < gc) p2 <<= 1;
        if (exact) {
            // classify the members; the tied ones go on a list (A.gidx is free while the run is sorted in shared memory)
            if (tid == 0) *s_cnt = 0;
            __syncthreads();
            for (int32_t base = warp * 32; base < gc; base += nwarps * 32) {
                const int32_t i = base + lane;
                const int32_t r = i < gc ? __ldcg(A.mem + gs + i) : -1;
                const bool act = r >= 0 && r != P.slot;
                unsigned long long h = KLPM_FAST_NOGROUP;
                if (act && !slot_done(R, A, r)) {
                    const FDyn d = ld_dyn(A.dyn + r);
                    const FStat s = ld_stat(A.stat + r);
                    if (d.pos == P.pos && d.ntok == P.ntok && d.m == P.m && d.m < s.len) __stcg(A.gidx + atomicAdd(s_cnt, 1), i);
                    else h = d.m < s.len ? group_hash(d.pos, d.ntok) : single_hash(r);
                }
                if (i < gc) { sh[i] = h; sr[i] = r; }
            }
            for (int32_t i = gc + tid; i < p2; i += nthr) { sh[i] = KLPM_FAST_NOGROUP; sr[i] = -1; }
            __syncthreads();
            // one tied member per warp at a time: compare it with the processed prompt's uncached tokens
            const int32_t nt = *s_cnt;
            for (int32_t k = warp; k < nt; k += nwarps) {
                const int32_t i = __ldcg(A.gidx + k);
                const int32_t r = sr[i];
                const FStat s = ld_stat(A.stat + r);
                const int32_t* qq = A.tok + s.soff;
                const int32_t lim = (s.len < P.len ? s.len : P.len) - P.m;
                const int32_t e = first_mismatch<true, 8>(qq + P.m, P.x + P.m, lim);
                if (lane == 0) {
                    const int32_t m2 = P.m + e;
                    const long long pos2 = P.vleaf + e - 1;
                    const int32_t ntok2 = m2 < s.len ? __ldg(qq + m2) : 0;
                    st_dyn_state(A.dyn + r, pos2, m2, ntok2);
                    if (A.lru) lru_move(A, r, __ldcg(reinterpret_cast<const int32_t*>(A.dyn + r) + 6), P.leaf);
                    const unsigned long long key = fast_key(m2, s.len, s.rank, A.score_mode);
                    __stcg(A.key + r, key);
                    if (R.skip) atomicOr(R.skip + (r >> 5), 1u << (r & 31));
                    if ((long long)r < P.admitted) atomicMax(R.t1 + (r >> A.lb_shift), key);
                    sh[i] = m2 < s.len ? group_hash(pos2, ntok2) : single_hash(r);
                }
            }
        } else {
            for (int32_t base = warp * 32; base < gc; base += nwarps * 32) {
                const int32_t i = base + lane;
                const int32_t r = i < gc ? __ldcg(A.mem + gs + i) : -1;
                bool touched;
                const unsigned long long h = fast_member(A, P, R, r, lane, &touched);
                if (i < gc) { __stcg(A.gh + i, (long long)h); __stcg(A.gidx + i, r); }
            }
            if (tid == 0) *s_cnt = 0;
        }
        __syncthreads();
        if (exact) {
            // regroup exactly: sort the members by the hash of their new group inside the run
            sort_and_group(A, R, sh, sr, gc, p2, gs);
        } else {
            // too many for the shared-memory sort: the same regrouping with the arrays in global memory
            sort_large_and_group(A, R, sh, sr, gc, gs);
        }
    }
    __syncthreads();
    tour_mid(R, warp, nwarps, lane);
    __syncthreads();
}

// The loop.  While arrivals are pending every decision is one careful step: admit who has arrived, pick from the
// tournament over all arrived slots (or the oldest slot), take the pick out of its leaf block, charge it and
// dissolve its group.  Once everybody has arrived the time of a pick no longer decides who can be picked, and the
// loop changes to list mode: all keys were sorted before the loop, so the longest-match pick is the next entry of
// that list that is still unprocessed and whose key has not changed since; the tournament is cut down to the slots
// whose key has changed (members of dissolved groups) and the pick is the larger of the two candidates.  A pick
// from the list touches no tournament at all, up to 32 decisions are made by one warp-wide step (up to 1,024 by a
// CTA-wide one, fast_batch_job), and the loop only records which slot each decision takes: the charge pass after the
// loop computes their outputs.
// G: some of the loop's bitmaps live in global memory (queues too long for shared memory).  The instance without them
// reads its bitmaps as plain shared-memory words.
template <bool G>
__global__ void __launch_bounds__(KLPM_FAST_THREADS, 1)
fast_run_kernel(FastArgs A) {
    extern __shared__ __align__(16) unsigned char fast_smem[];
    __shared__ FastJob s_job;
    __shared__ int s_cnt;
    __shared__ int32_t s_H[32], s_E[32];      // a batch's oldest-first and longest-match picks, by rank
    __shared__ FastBatchIO s_bio;             // a CTA-wide batch: what the sequencer hands over and gets back
    __shared__ int32_t s_scan[KLPM_FAST_THREADS / 32];
    __shared__ TreeState s_st;                // trees with a budget: the tree's counters while the loop runs
    __shared__ int32_t s_memcur;              // trees with a budget: first free entry of the member array
    __shared__ unsigned int s_dirty[256];
    if (A.lru && *reinterpret_cast<const volatile int32_t*>(A.skip)) return;       // the capacity check said no: nothing is touched
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    const int32_t n = A.n;
    const int32_t nb1p = (A.nb + 31) & ~31, n2 = nb1p >> 5, n2p = (n2 + 31) & ~31, n3 = n2p >> 5;
    const int32_t nwords = (n + 31) >> 5;
    FastTour R;
    R.t1 = reinterpret_cast<unsigned long long*>(fast_smem);
    R.t2 = R.t1 + nb1p;
    R.t3 = R.t2 + n2p;
    R.n2 = n2; R.n3 = n3;
    unsigned long long* sh = R.t3 + 32;
    int32_t* sr = reinterpret_cast<int32_t*>(sh + KLPM_FAST_SORT_CAP);
    unsigned int* s_bits = reinterpret_cast<unsigned int*>(sr + KLPM_FAST_SORT_CAP);
    // the bitmaps: in shared memory while they fit, in global memory (cleared / filled by the host side) otherwise
    R.g_done = A.done_in_smem ? 0 : 1;
    R.g_bits = A.bits_in_smem ? 0 : 1;
    R.done = A.done_in_smem ? s_bits : A.done;
    R.skip = !A.list_mode ? nullptr : A.bits_in_smem ? s_bits + nwords : A.gskip;
    R.gb = !A.list_mode ? nullptr : A.bits_in_smem ? s_bits + 2 * nwords : A.gbits;
    R.dirty = s_dirty;
    unsigned int* const s_done = R.done;
    if (!G) { R.g_done = 0; R.g_bits = 0; }
    const int gdone = G ? R.g_done : 0, gbits = G ? R.g_bits : 0;
    for (int32_t i = threadIdx.x; i < nb1p + n2p + 32; i += blockDim.x) R.t1[i] = 0ULL;
    if (threadIdx.x == 0) { s_memcur = A.lru ? 2 * n : n; if (A.lru) s_st = *A.st; }
    if (A.done_in_smem) for (int32_t i = threadIdx.x; i < nwords; i += blockDim.x) s_bits[i] = 0u;
    if (A.list_mode && A.bits_in_smem) for (int32_t i = threadIdx.x; i < nwords; i += blockDim.x) { R.skip[i] = 0u; R.gb[i] = __ldcg(A.gbits + i); }
    __syncthreads();

    if (warp != 0) {
        for (;;) {
            named_bar(1, KLPM_FAST_THREADS);
            const FastJob J = s_job;
            if (J.type == FAST_JOB_EXIT) return;
            if (J.type == FAST_JOB_BATCH) { fast_batch_job<G>(A, R, &s_bio, sr, sr + 1024, sr + 2048, reinterpret_cast<int32_t*>(sh), s_scan, nwords); continue; }
            fast_job(A, R, J, sh, sr, &s_cnt, &s_memcur);
        }
    }

    // ---------------------------------------------------------------- the sequencer (warp 0)
    const long long INF = 0x7fffffffffffffffLL;
    long long now = A.start_tick;
    int32_t head = 0, admitted = 0;
    long long next_t = __ldg(&A.stat[0].t);
    unsigned long long root = 0;
    long long n_careful = 0, n_cta_dissolve = 0, n_scan = 0, n_evict = 0, cy_tree = 0, cy_scan = 0, cy_dissolve = 0;
    int32_t cyc = 0;                                        // c mod k
    int32_t c = 0;
    bool failed = false;

    // first unprocessed slot at or after `head` (which is processed)
    auto advance_head = [&]() {
        if (head + 1 < n) {                                 // the usual cases: the next slot, or one of the next 32 to 63
            const int32_t h1 = head + 1, wi = h1 >> 5;
            const unsigned f0 = ~bm_ld(s_done, wi, gdone) & ~((1u << (h1 & 31)) - 1u);
            if (f0) { head = wi * 32 + __ffs(f0) - 1; if (head > n) head = n; return; }
            if (wi + 1 < nwords) {
                const unsigned f1 = ~bm_ld(s_done, wi + 1, gdone);
                if (f1) { head = (wi + 1) * 32 + __ffs(f1) - 1; if (head > n) head = n; return; }
            }
        }
        int32_t w0 = head >> 5;
        for (;;) {
            const int32_t wi = w0 + lane;
            unsigned w = 0u;                                  // past the end: "unprocessed", so the search stops
            if (wi < nwords) w = bm_ld(s_done, wi, gdone);
            if (wi == (head >> 5)) w |= (1u << (head & 31)) - 1u;
            const unsigned bal = __ballot_sync(FULL_MASK, w != 0xffffffffu);
            if (bal) {
                const int src = __ffs(bal) - 1;
                const unsigned fw = ~__shfl_sync(FULL_MASK, w, src);
                head = (w0 + src) * 32 + __ffs(fw) - 1;
                break;
            }
            w0 += 32;
        }
        if (head > n) head = n;
    };
    // slot j is processed from now on (every lane performs the same shared-memory stores)
    auto mark_done = [&](int32_t j) {
        if (!gdone) s_done[j >> 5] |= 1u << (j & 31);
        else if (lane == 0) __stcg(s_done + (j >> 5), __ldcg(s_done + (j >> 5)) | (1u << (j & 31)));
        if (R.skip) {
            if (!gbits) R.skip[j >> 5] |= 1u << (j & 31);
            else if (lane == 0) __stcg(R.skip + (j >> 5), __ldcg(R.skip + (j >> 5)) | (1u << (j & 31)));
        }
        __syncwarp();
    };
    // Charge pick `slot` (Definition 2), write its outputs, and let the queries tied with it match into its new
    // leaf.  The caller has taken the slot out of the tournament or the list and marked it processed.
    auto careful = [&](int32_t slot, bool charge, const FDyn& d, const FStat& s) {
        const int32_t m = d.m, len = s.len, unc = len - m;
        if (charge) {
            const long long begin = now > s.t ? now : s.t;
            const long long Rj = begin + (A.c_den + A.c_num * (long long)len) * (long long)unc;
            now = Rj;
            if (lane == 0) {
                if (A.order) A.order[c] = s.ord;
                A.uncached[s.ord] = unc; A.ttft[s.ord] = Rj - s.t;
                if (A.completion) A.completion[s.ord] = Rj;
            }
        } else if (lane == 0) {
            A.order[c] = slot;                              // list mode: the charge pass after the loop does the rest
        }
        // the new leaf's positions: unique per decision, above every real pool index
        const long long vleaf = A.vbase + ((long long)c << 32);
        ++c;
        int32_t leaf = -1;
        ++n_careful;
        if (A.lru) {
            const long long t_tree = clock64();
            // ---- the tree's node arrays follow the decision (what insert_serial does, minus the child table and the
            //      tokens, which the pass after the loop writes for the nodes that are still alive then)
            const TreeDev& T = A.T;
            if (lane == 0) atomicSub(A.parked + d.hint, 1);
            if (s_st.clock + 1 >= T.max_clock || s_st.n_nodes + 2 > T.max_nodes) {        // (the check before the loop rules this out)
                if (lane == 0) set_status(A.st, RT_ERR_CAPACITY, 114);
                failed = true; return;
            }
            const long long clock = s_st.clock + 1;
            // Two chains of dependent loads are started side by side: the node the match ends in (hint, then up), and
            // the least recently used leaf (the cursor's next 32 clock values, their owners' fields) -- most decisions
            // evict, and which leaf goes does not depend on the pick, except that the node stamped below is safe.
            const long long cur0 = s_st.lru_cursor;
            int32_t a = d.hint;
            int32_t ds = T.depth_start[a], sl = T.span_len[a], pa = T.parent[a];
            const long long pre_cc = cur0 + lane;
            const int32_t pre_v = pre_cc < clock ? T.clock_owner[pre_cc] : 0;
            bool pre_ok = false;
            int32_t pre_P = 0, pre_len = 0, pre_parked = 0;
            if (pre_v > 0) {
                pre_ok = !T.dead[pre_v] && T.last_access[pre_v] == pre_cc && T.nchild[pre_v] == 0;
                pre_P = T.parent[pre_v]; pre_len = T.span_len[pre_v]; pre_parked = __ldcg(A.parked + pre_v);
            }
            while (a != 0 && m <= ds) { a = pa; ds = T.depth_start[a]; sl = T.span_len[a]; pa = T.parent[a]; }
            const int32_t o = a == 0 ? 0 : m - ds;
            int32_t end = a;
            bool cut = false;
            long long n_nodes = s_st.n_nodes, live_nodes = s_st.live_nodes, tokens_live = s_st.tokens_live, evictions = s_st.evictions;
            if (a != 0 && o < sl) {                         // node boundary inside a's edge: a new node takes the upper part
                const int32_t u = (int32_t)n_nodes++;
                ++live_nodes;
                cut = true;
                if (lane == 0) {
                    const int64_t so = T.span_off[a];
                    T.parent[u] = pa; T.depth_start[u] = ds; T.span_off[u] = so; T.span_len[u] = o;
                    T.nchild[u] = 1; T.dead[u] = 0; T.last_access[u] = T.last_access[a];
                    T.span_off[a] = so + o; T.span_len[a] = sl - o; T.depth_start[a] = ds + o; T.parent[a] = u;
                }
                end = u;
            }
            if (end != 0 && lane == 0) { T.last_access[end] = clock; T.clock_owner[clock] = end; }
            __syncwarp();
            // least recently used leaves go until the prompt's uncached tokens fit (the node just stamped is safe)
            bool scan = false;
            int32_t small_v[8];                             // evicted leaves whose parked queries this warp looks after itself
            int n_small = 0;
            long long cur = cur0;
            // The leaves of the window that was loaded ahead are taken one after the other while the window's view of who
            // is a leaf holds: it ends when an eviction turns a parent into a leaf (that parent may be the next to go).
            bool first = true, win_ok = true;
            unsigned win = 0;
            while (tokens_live + unc > T.budget) {
                int32_t victim = -1, P = 0, vlen = 0, vparked = 0;
                if (win_ok) {
                    if (first) { win = __ballot_sync(FULL_MASK, pre_ok && pre_v != end); first = false; }      // (the node stamped above has moved on)
                    if (win) {
                        const int src = __ffs(win) - 1;
                        win &= win - 1;
                        victim = __shfl_sync(FULL_MASK, pre_v, src); P = __shfl_sync(FULL_MASK, pre_P, src);
                        vlen = __shfl_sync(FULL_MASK, pre_len, src); vparked = __shfl_sync(FULL_MASK, pre_parked, src);
                        cur = cur0 + src;
                        if (cut && victim == a) { P = T.parent[victim]; vlen = T.span_len[victim]; }      // the lower part of the edge just cut
                    } else {
                        cur = cur0 + 32;
                        win_ok = false;
                    }
                }
                if (victim < 0) {
                    while (cur < clock) {                   // 32 clock values at a time
                        const long long cc = cur + lane;
                        const int32_t v = cc < clock ? T.clock_owner[cc] : 0;
                        const bool ok = v > 0 && !T.dead[v] && T.last_access[v] == cc && T.nchild[v] == 0;
                        const unsigned bal = __ballot_sync(FULL_MASK, ok);
                        if (bal) { const int src = __ffs(bal) - 1; victim = __shfl_sync(FULL_MASK, v, src); cur += src; break; }
                        cur += 32;
                    }
                    if (victim >= 0) { P = T.parent[victim]; vlen = T.span_len[victim]; vparked = __ldcg(A.parked + victim); }
                }
                if (victim < 0) {
                    if (lane == 0) set_status(A.st, RT_ERR_BUDGET);
                    failed = true; break;
                }
                tokens_live -= vlen;
                --live_nodes; ++evictions; ++n_evict;
                if (vparked > 0) {
                    // Queries are parked in the evicted leaf.  If one run of the member array is known to hold every slot
                    // whose hint is this leaf, the warp looks after them itself below (up to 8 such leaves and 32 slots
                    // that fall back per decision); otherwise the whole CTA scans the unprocessed slots.
                    const int2 lr = __ldcg(A.leaf_run + victim);
                    if (lr.y > 0 && lr.y <= 1024 && n_small < 8) { small_v[n_small] = victim; ++n_small; }
                    else scan = true;
                }
                int new_leaf = 0;
                if (lane == 0) {
                    T.dead[victim] = 1;
                    const int32_t nc = T.nchild[P] - 1;
                    T.nchild[P] = nc;
                    const long long stamp = T.last_access[victim];
                    if (P != 0 && stamp >= T.last_access[P]) { T.last_access[P] = stamp; T.clock_owner[stamp] = P; }
                    new_leaf = nc == 0 && P != 0;
                }
                __syncwarp();
                if (win_ok && __shfl_sync(FULL_MASK, new_leaf, 0)) win_ok = false;
            }
            if (cur > clock) cur = clock;
            if (!failed && unc > 0) {
                leaf = (int32_t)n_nodes++;
                ++live_nodes;
                tokens_live += unc;
                if (lane == 0) {
                    T.parent[leaf] = end; T.depth_start[leaf] = m; T.span_off[leaf] = vleaf; T.span_len[leaf] = unc;
                    T.nchild[leaf] = 0; T.dead[leaf] = 0; T.last_access[leaf] = clock; T.clock_owner[clock] = leaf;
                    T.nchild[end]++;
                    A.leaf_run[leaf] = make_int2(d.gstart, d.gcount);     // whoever gets parked in it is a member of the pick's group
                }
            }
            __syncwarp();
            if (lane == 0) {
                s_st.clock = clock; s_st.n_nodes = n_nodes; s_st.live_nodes = live_nodes; s_st.tokens_live = tokens_live;
                s_st.evictions = evictions; s_st.lru_cursor = cur;
            }
            __syncwarp();
            // ---- evicted leaves whose parked queries sit in known member runs: the warp moves them itself.  All leaves of
            //      this decision are taken together: two of them, one above the other, send their queries to one group.
            if (n_small > 0 && !scan && !failed) {
                // first pass: how many slots fall back (more than 32: leave it to the scan)
                int32_t n_fall = 0;
                for (int sv = 0; sv < n_small; ++sv) {
                    const int32_t v = small_v[sv];
                    const int2 lr = __ldcg(A.leaf_run + v);
                    const int32_t ds_v = T.depth_start[v];
                    for (int32_t base = 0; base < lr.y; base += 32) {
                        const int32_t r = base + lane < lr.y ? __ldcg(A.mem + lr.x + base + lane) : -1;
                        bool hit = r >= 0 && !slot_done(R, A, r) && __ldcg(A.hintc + r) == v;
                        if (hit) hit = __ldcg(reinterpret_cast<const int32_t*>(A.dyn + r) + 2) > ds_v;
                        const unsigned same = __match_any_sync(FULL_MASK, hit ? r : -1 - lane);       // a slot can be listed twice in a run
                        if (hit && (int)(__ffs(same) - 1) != lane) hit = false;
                        n_fall += __popc(__ballot_sync(FULL_MASK, hit));
                    }
                }
                if (n_fall > 32) scan = true;
            }
            if (n_small > 0 && !scan && !failed) {
                // second pass: every member whose hint is a dead leaf walks up; those that lose tokens are collected
                int32_t f_slot = -1;                        // lane k holds the k-th slot that fell back
                unsigned long long f_hash = KLPM_FAST_NOGROUP;
                int32_t n_f = 0;
                for (int sv = 0; sv < n_small; ++sv) {
                    const int32_t v = small_v[sv];
                    const int2 lr = __ldcg(A.leaf_run + v);
                    for (int32_t base = 0; base < lr.y; base += 32) {
                        const int32_t r = base + lane < lr.y ? __ldcg(A.mem + lr.x + base + lane) : -1;
                        bool hit = r >= 0 && !slot_done(R, A, r) && __ldcg(A.hintc + r) == v;
                        const unsigned same = __match_any_sync(FULL_MASK, hit ? r : -1 - lane);
                        if (hit && (int)(__ffs(same) - 1) != lane) hit = false;
                        bool fell = false;
                        unsigned long long h = KLPM_FAST_NOGROUP;
                        if (hit) {
                            const int32_t m0 = __ldcg(reinterpret_cast<const int32_t*>(A.dyn + r) + 2);
                            int32_t mm = m0, a = v;
                            while (a != 0) {
                                const bool dead = T.dead[a] != 0;
                                const int32_t dsa = T.depth_start[a];
                                if (dead) { if (dsa < mm) mm = dsa; }
                                else if (mm > dsa) break;
                                a = T.parent[a];
                            }
                            st_dyn_hint(A.dyn + r, a);
                            __stcg(A.hintc + r, a);
                            atomicAdd(A.parked + a, 1);
                            A.leaf_run[a].y = -1;
                            if (mm != m0) {
                                const FStat fs = ld_stat(A.stat + r);
                                const long long pos = a == 0 ? -1 : T.span_off[a] + (long long)(mm - T.depth_start[a]) - 1;
                                const int32_t ntok = __ldg(A.tok + fs.soff + mm);
                                st_dyn_state(A.dyn + r, pos, mm, ntok);
                                __stcg(A.key + r, fast_key(mm, fs.len, fs.rank, A.score_mode));
                                h = group_hash(pos, ntok);
                                fell = true;
                            }
                        }
                        const unsigned fb = __ballot_sync(FULL_MASK, fell);
                        const int32_t my = n_f + __popc(fb & ((1u << lane) - 1u));
                        for (unsigned bits = fb; bits; bits &= bits - 1) {      // hand each fallen slot to the lane that keeps it
                            const int src = __ffs(bits) - 1;
                            const int32_t dst = __shfl_sync(FULL_MASK, my, src);
                            const int32_t rr = __shfl_sync(FULL_MASK, r, src);
                            const unsigned long long hh = __shfl_sync(FULL_MASK, h, src);
                            if (lane == dst) { f_slot = rr; f_hash = hh; }
                        }
                        n_f += __popc(fb);
                        __syncwarp();
                    }
                }
                if (n_f > 0) {
                    // the fallen slots are grouped afresh in a run appended to the member array (ranked by shuffles)
                    const int32_t base = s_memcur;
                    if ((long long)base + n_f > (long long)A.mem_cap) {
                        if (lane == 0) set_status(A.st, RT_ERR_CAPACITY, 113);
                        failed = true;
                    } else {
                        int32_t rank = 0, start = 0, cnt = 0;
                        for (int k2i = 0; k2i < 32; ++k2i) {
                            const unsigned long long hk = __shfl_sync(FULL_MASK, f_hash, k2i);
                            const bool lt = hk < f_hash, eq = hk == f_hash;
                            start += lt; cnt += eq; rank += (lt || (eq && k2i < lane));
                        }
                        if (f_slot >= 0) {
                            __stcg(A.mem + base + rank, f_slot);
                            st_dyn_group(A.dyn + f_slot, base + start, cnt);
                            set_grouped(R, f_slot, cnt > 1);
                        }
                        if (lane == 0) s_memcur = base + n_f;
                        __syncwarp();
                        // their keys went down: the leaf blocks of the arrived ones are recomputed
                        for (int k2i = 0; k2i < n_f; ++k2i) {
                            const int32_t rr = __shfl_sync(FULL_MASK, f_slot, k2i);
                            if (rr < admitted) {
                                const int32_t bb = rr >> A.lb_shift;
                                admit_blocks_one(A, R, bb, bb << A.lb_shift, admitted, lane);
                                __syncwarp();
                                root = tour_update(R, bb, lane);
                            }
                        }
                    }
                }
            }
            cy_tree += clock64() - t_tree;
            if (scan) {                                     // somebody was parked in an evicted leaf
                const long long t_scan = clock64();
                ++n_scan;
                if (lane == 0) { s_job.type = FAST_JOB_FALLBACK; s_job.a0 = head < slot ? head : slot; s_job.a1 = admitted; }
                __threadfence_block();
                __syncwarp();
                named_bar(1, KLPM_FAST_THREADS);
                const FastJob J = s_job;
                fast_job(A, R, J, sh, sr, &s_cnt, &s_memcur);
                root = tour_top(R, lane);
                cy_scan += clock64() - t_scan;
            }
            if (failed) return;
        }
        if (unc > 0 && d.gcount > 1) {
            FastPick P;
            P.slot = slot; P.m = m; P.len = len; P.ntok = d.ntok; P.x = A.tok + s.soff; P.pos = d.pos; P.vleaf = vleaf;
            P.admitted = admitted; P.gstart = d.gstart; P.gcount = d.gcount; P.leaf = leaf;
            // small groups are handled by this warp alone, unless several long compares are better spread over the CTA
            if (d.gcount <= 32 && !(d.gcount > 2 && unc > 512)) {
                const int32_t r = lane < d.gcount ? __ldcg(A.mem + d.gstart + lane) : -1;
                bool touched;
                const unsigned long long h = fast_member(A, P, R, r, lane, &touched);
                int32_t rank = 0, start = 0, cnt = 0;       // regroup inside the run
                for (int k2i = 0; k2i < 32; ++k2i) {
                    const unsigned long long hk = __shfl_sync(FULL_MASK, h, k2i);
                    const bool lt = hk < h, eq = hk == h;
                    start += lt; cnt += eq; rank += (lt || (eq && k2i < lane));
                }
                if (h != KLPM_FAST_NOGROUP) {
                    __stcg(A.mem + d.gstart + rank, r);
                    st_dyn_group(A.dyn + r, d.gstart + start, cnt);
                    set_grouped(R, r, cnt > 1);
                }
                __syncwarp();
                unsigned tm = __ballot_sync(FULL_MASK, touched);
                while (tm) {
                    const int src = __ffs(tm) - 1; tm &= tm - 1;
                    const int32_t bb = __shfl_sync(FULL_MASK, r >> A.lb_shift, src);
                    root = tour_update(R, bb, lane);
                }
            } else {
                const long long t_dis = clock64();
                ++n_cta_dissolve;
                if (lane == 0) { s_job.type = FAST_JOB_DISSOLVE; s_job.pick = P; }
                __syncwarp();
                named_bar(1, KLPM_FAST_THREADS);
                const FastJob J = s_job;
                fast_job(A, R, J, sh, sr, &s_cnt, &s_memcur);
                root = tour_top(R, lane);
                cy_dissolve += clock64() - t_dis;
            }
        }
    };

    // ================================================================ a given order (klpm_replay): no admission, no pick
    if (A.fixed) {
        const int32_t nfix = *reinterpret_cast<const volatile int32_t*>(A.n_fixed);
        while (c < nfix && !failed) {
            const int32_t slot = __ldg(A.fixed + c);        // slots are the queries in index order here
            const FDyn pd = ld_dyn(A.dyn + slot);
            const FStat ps = ld_stat(A.stat + slot);
            mark_done(slot);
            careful(slot, true, pd, ps);                     // (head stays 0 and nobody is admitted: scans cover every slot)
            __syncwarp();
        }
        c = n;                                               // nothing is left for the policy loops below
    }

    // everybody is waiting as the loop starts: no arrival will ever have to be admitted
    if (A.list_mode && __ldg(&A.stat[n - 1].t) <= now) { admitted = n; next_t = INF; }

    // ================================================================ arrivals pending: one careful step per decision
    while (c < n && !failed && !(A.list_mode && admitted == n)) {
        // ---- time and arrivals: idle until somebody has arrived, then admit everybody who has
        if (head == admitted && next_t > now) now = next_t;
        if (next_t <= now) {
            int32_t a1 = admitted;
            {
                const long long r = (long long)a1 + lane;
                const bool in = r < n && __ldg(&A.stat[r].t) <= now;
                const unsigned bal = __ballot_sync(FULL_MASK, in);
                const int cnt = bal == FULL_MASK ? 32 : __ffs(~bal) - 1;
                a1 += cnt;
                if (cnt == 32 && a1 < n) {                 // a full window: gallop, then bisect (lane 0)
                    long long lo = a1, hi = n;
                    if (lane == 0 && __ldg(&A.stat[lo].t) <= now) {
                        long long step = 1;
                        ++lo;
                        while (lo + step <= hi && __ldg(&A.stat[lo + step - 1].t) <= now) { lo += step; step <<= 1; }
                        if (lo + step < hi) hi = lo + step;
                        while (lo < hi) { const long long mid = (lo + hi) >> 1; if (__ldg(&A.stat[mid].t) <= now) lo = mid + 1; else hi = mid; }
                    }
                    a1 = (int32_t)__shfl_sync(FULL_MASK, lo, 0);
                }
            }
            if (a1 - admitted <= 32) {
                const int32_t r = admitted + lane;
                if (r < a1) atomicMax(R.t1 + (r >> A.lb_shift), __ldcg(A.key + r));
                __syncwarp();
                root = tour_update(R, admitted >> A.lb_shift, lane);
                if (((a1 - 1) >> A.lb_shift) != (admitted >> A.lb_shift)) root = tour_update(R, (a1 - 1) >> A.lb_shift, lane);
            } else {
                if (lane == 0) { s_job.type = FAST_JOB_ADMIT; s_job.a0 = admitted; s_job.a1 = a1; }
                __syncwarp();
                named_bar(1, KLPM_FAST_THREADS);
                const FastJob J = s_job;
                fast_job(A, R, J, sh, sr, &s_cnt, &s_memcur);
                root = tour_top(R, lane);
            }
            admitted = a1;
            next_t = admitted < n ? __ldg(&A.stat[admitted].t) : INF;
        }
        // ---- pick
        const bool fcfs_turn = A.policy == KLPM_POLICY_FCFS || (A.policy == KLPM_POLICY_KLPM && cyc == 0);
        if (++cyc == A.k) cyc = 0;
        int32_t slot = head;
        if (!fcfs_turn) {
            const unsigned rk = 0xffffffffu - (unsigned)(root & 0xffffffffULL);
            slot = A.pinv ? __ldg(A.pinv + rk) : (int32_t)rk;
        }
        if (slot < 0 || slot >= admitted || slot_done(R, A, slot)) { if (lane == 0) set_status(A.st, RT_ERR_LIMIT, 105); failed = true; break; }   // cannot happen
        // ---- the pick leaves its leaf block (its two records are asked for first: they travel with the block's keys)
        const FDyn pd = ld_dyn(A.dyn + slot);
        const FStat ps = ld_stat(A.stat + slot);
        const int32_t b = slot >> A.lb_shift;
        unsigned long long bm = 0;
        for (int32_t u = lane; u < (1 << A.lb_shift); u += 32) {
            const long long r = ((long long)b << A.lb_shift) + u;
            if (r < admitted && r != slot && !slot_done(R, A, r)) { const unsigned long long kk = __ldcg(A.key + r); if (kk > bm) bm = kk; }
        }
        root = tour_set(R, b, warp_max64r(bm), lane);
        mark_done(slot);
        careful(slot, true, pd, ps);
        if (slot == head) advance_head();
        __syncwarp();
    }

    // ================================================================ list mode
    if (c < n && !failed) {
        if (lane == 0) s_job.type = FAST_JOB_REBUILD;
        __syncwarp();
        named_bar(1, KLPM_FAST_THREADS);
        {
            const FastJob J = s_job;
            fast_job(A, R, J, sh, sr, &s_cnt, &s_memcur);
        }
        root = tour_top(R, lane);
        // the sorted list, 32 entries at a time: lane l holds entry (cur & ~31) + l, the next 32 are on their way
        int32_t cur = 0;
        auto window = [&](int32_t base, long long* wk_, int32_t* ws_) {
            const long long i = (long long)base + lane;
            *wk_ = i < n ? __ldg(A.lk + i) : INF;
            *ws_ = i < n ? __ldg(A.ls + i) : -1;
        };
        long long wk, nk; int32_t ws, ns;
        window(0, &wk, &ws);
        window(32, &nk, &ns);
        auto advance_cur = [&]() {
            ++cur;
            if ((cur & 31) == 0) { wk = nk; ws = ns; window(cur + 32, &nk, &ns); }
        };
        // From here on the time of a decision influences no decision, so the loop only records which slot each
        // decision takes (in `order`); the charge pass after the loop turns that into query indices, uncached tokens,
        // completion times and TTFTs (Definition 2 with R_prev >= t_j is a running sum of the costs).
        if (lane == 0) { A.post->c0 = c; A.post->now0 = now; }
        int32_t myj = 0;
        // Up to 32 decisions at once.  As long as nothing interferes, the coming longest-match picks are the next
        // entries of the list that still count and the coming oldest-first picks are the next unprocessed slots,
        // interleaved as the policy says.  The warp gathers both sets side by side and checks that they cannot
        // have influenced each other: no slot in both (a list entry inside the range of slots the oldest-first
        // picks consume), none whose group has other members, none whose key sits in the tournament, and the
        // tournament's root below the smallest key taken from the list.  The batch is cut before the first decision
        // that fails a check; then lane i makes decision c + i.  If fewer than two decisions are left that way,
        // nothing has been changed and the next decisions are made one at a time below.
        const int32_t lane_div_k = lane / A.k;              // y / k for y = 0..31, looked up by shuffle
        bool tb_cut = false;                                // the last warp-wide step stopped before a decision it could not take
        auto try_batch = [&]() -> bool {
            // oldest-first turns among the next x decisions, for x = lane (f_lo) and x = lane + 1 (f_hi): under k-LPM
            // the first such turn is decision i0 = (k - cyc) mod k, then every k-th
            int32_t f_lo, f_hi;
            if (A.policy == KLPM_POLICY_FCFS) { f_lo = lane; f_hi = lane + 1; }
            else if (A.policy == KLPM_POLICY_LPM) { f_lo = 0; f_hi = 0; }
            else {
                const int32_t i0 = cyc == 0 ? 0 : A.k - cyc;
                const int32_t y_lo = lane - i0 - 1, y_hi = lane - i0;
                const int32_t q_lo = __shfl_sync(FULL_MASK, lane_div_k, y_lo > 0 ? y_lo : 0);
                const int32_t q_hi = __shfl_sync(FULL_MASK, lane_div_k, y_hi > 0 ? y_hi : 0);
                f_lo = y_lo >= 0 ? q_lo + 1 : 0;
                f_hi = y_hi >= 0 ? q_hi + 1 : 0;
            }
            // the list entries cur .. cur + 31 (in this window or the next) that still count
            long long kk; int32_t es; unsigned mask;
            {
                const int32_t off = (cur & 31) + lane;
                const long long k0 = __shfl_sync(FULL_MASK, wk, off & 31), k1 = __shfl_sync(FULL_MASK, nk, off & 31);
                const int32_t s0 = __shfl_sync(FULL_MASK, ws, off & 31), s1 = __shfl_sync(FULL_MASK, ns, off & 31);
                kk = off < 32 ? k0 : k1;
                es = off < 32 ? s0 : s1;
                const bool valid = (long long)cur + lane < n;
                mask = __ballot_sync(FULL_MASK, valid && !((bm_ld(R.skip, es >> 5, gbits) >> (es & 31)) & 1u));
            }
            // as many decisions as those entries allow: lane x asks whether x + 1 decisions need no more of them
            const int32_t avail = __popc(mask);
            const int32_t B0 = __popc(__ballot_sync(FULL_MASK, c + lane < n && (lane + 1) - f_hi <= avail));
            if (B0 < 2) return false;
            const int32_t nF0 = __shfl_sync(FULL_MASK, f_hi, B0 - 1), nL0 = B0 - nF0;
            // the next nF0 unprocessed slots; limF = how many of them can be taken before one needs the careful step
            int32_t hs = -1, hmax0 = -1, limF = nF0;
            if (nF0 > 0) {
                const int32_t w0 = head >> 5;
                const int32_t qk = lane < nF0 ? lane : nF0 - 1;       // lane q looks for the q-th unprocessed slot
                auto free_word = [&](int32_t wi) -> unsigned {        // unprocessed slots of bitmap word wi, from head on
                    unsigned w = wi < nwords ? bm_ld(s_done, wi, gdone) : 0xffffffffu;
                    if (wi == nwords - 1 && (n & 31)) w |= ~((1u << (n & 31)) - 1u);
                    if (wi == w0) w |= (1u << (head & 31)) - 1u;
                    return ~w;
                };
                const unsigned f0 = free_word(w0), f1 = free_word(w0 + 1);
                const int32_t c0 = __popc(f0);
                if (c0 + __popc(f1) >= nF0) {                         // the usual case: they are all in the first two words
                    hs = qk < c0 ? w0 * 32 + kth_set_bit(f0, qk + 1) : (w0 + 1) * 32 + kth_set_bit(f1, qk - c0 + 1);
                } else {                                              // up to 32 words: running counts, then a search per lane
                    const unsigned fr = free_word(w0 + lane);
                    const int32_t cnt = __popc(fr);
                    int32_t inc = cnt;
#pragma unroll
                    for (int dlt = 1; dlt < 32; dlt <<= 1) { const int32_t o = __shfl_up_sync(FULL_MASK, inc, dlt); if (lane >= dlt) inc += o; }
                    if (__shfl_sync(FULL_MASK, inc, 31) < nF0) return false;
                    int L = 0;
#pragma unroll
                    for (int step = 16; step > 0; step >>= 1) if (__shfl_sync(FULL_MASK, inc, L + step - 1) <= qk) L += step;
                    const unsigned frL = __shfl_sync(FULL_MASK, fr, L);
                    const int32_t preL = __shfl_sync(FULL_MASK, inc - cnt, L);
                    hs = (w0 + L) * 32 + kth_set_bit(frL, qk - preL + 1);
                }
                hmax0 = __shfl_sync(FULL_MASK, hs, nF0 - 1);
                // its key sits in the tournament, or its group has other members
                const unsigned badH = __ballot_sync(FULL_MASK, lane < nF0 && ((((bm_ld(R.skip, hs >> 5, gbits) | bm_ld(R.gb, hs >> 5, gbits)) >> (hs & 31)) & 1u)));
                if (badH) limF = __ffs(badH) - 1;
            }
            // limL = how many list entries can be taken before one is grouped, could also be an oldest-first pick of
            // this batch, or has a key below the tournament's root
            const bool ok = (mask >> lane) & 1u;
            const int32_t rank = __popc(mask & ((1u << lane) - 1u));
            int32_t limL = nL0;
            int32_t soft = -1;                              // slot of the entry that stops the batch, if it is only suspected of being an oldest-first pick too
            {
                const unsigned long long ek = ~((unsigned long long)kk ^ 0x8000000000000000ULL);
                const bool hard = (((bm_ld(R.gb, es >> 5, gbits) >> (es & 31)) & 1u)) || root > ek;
                const unsigned badE = __ballot_sync(FULL_MASK, ok && rank < nL0 && (hard || (es >= head && es <= hmax0)));
                if (badE) {
                    const int src = __ffs(badE) - 1;
                    limL = __popc(mask & ((1u << src) - 1u));
                    if (!__shfl_sync(FULL_MASK, (int)hard, src)) soft = __shfl_sync(FULL_MASK, es, src);
                }
            }
            int32_t B = __popc(__ballot_sync(FULL_MASK, lane < B0 && f_hi <= limF && (lane + 1) - f_hi <= limL));
            if (soft >= 0 && B < B0 && B < 32) {
                // the decision after the batch (lane B's): if it is the longest-match turn that takes that entry and the
                // oldest-first picks made until then all lie before its slot, it becomes the batch's last decision
                const int32_t fl = __shfl_sync(FULL_MASK, f_lo, B), fh = __shfl_sync(FULL_MASK, f_hi, B);
                const int32_t last_h = __shfl_sync(FULL_MASK, hs, fl > 0 ? fl - 1 : 0);
                if (fh == fl && B - fl == limL && fl <= limF && (fl == 0 || last_h < soft)) { ++B; ++limL; }
            }
            if (B < 2) return false;
            tb_cut = B < B0 && soft < 0;
            const int32_t nF = __shfl_sync(FULL_MASK, f_hi, B - 1), nL = B - nF;
            const int32_t hmax = nF > 0 ? __shfl_sync(FULL_MASK, hs, nF - 1) : -1;
            if (lane < nF) s_H[lane] = hs;
            int32_t consumed = 0;
            if (nL > 0) {
                consumed = kth_set_bit(mask, nL) + 1;
                if (ok && rank < nL) s_E[rank] = es;
            }
            __syncwarp();
            // commit: lane i makes decision c + i
            if (lane < B) {
                myj = f_hi > f_lo ? s_H[f_lo] : s_E[lane - f_lo];
                atomicOr(s_done + (myj >> 5), 1u << (myj & 31));
                atomicOr(R.skip + (myj >> 5), 1u << (myj & 31));
            }
            __syncwarp();
            if (lane < B) A.order[c + lane] = myj;
            c += B;
            if (A.policy == KLPM_POLICY_KLPM) cyc = (cyc + B) % A.k;
            if (consumed) {
                const int32_t ncur = cur + consumed;
                if ((ncur >> 5) != (cur >> 5)) { wk = nk; ws = ns; window((ncur & ~31) + 32, &nk, &ns); }
                cur = ncur;
            }
            if (nF > 0) { head = hmax; advance_head(); }
            else if (head < n && ((bm_ld(s_done, head >> 5, gdone) >> (head & 31)) & 1u)) advance_head();
            return true;
        };
        int32_t vb_wait = 0, vb_back = 1;                   // decisions until the next attempt; doubles while attempts fail
        int32_t cb_wait = 0, cb_back = 8;                   // the same for the CTA-wide batch (loop iterations; 8 .. 1,024)
        int32_t cb_until = 0, cb_fail = 0;                  // after an attempt that made no decision: not before decision cb_until; attempts failed in a row
        int32_t calm = KLPM_FAST_CALM;                      // consecutive full warp-wide steps: the CTA-wide batch is tried in calm water only
        long long n_cta_try = 0, n_cta_ok = 0, dec_cta = 0, n_warp_ok = 0, dec_warp = 0, dec_one = 0, cy_cta = 0, cy_warp = 0;
        // a batch that was cut short stopped before a decision only the one-at-a-time path can take: that one comes
        // next, without another attempt that would find it again
        bool one_next = false;
        while (c < n && !failed) {
            // first choice: the whole CTA makes up to 1,024 decisions (the sort scratch is free between dissolves)
            if (!one_next && cb_wait <= 0 && calm >= KLPM_FAST_CALM && c >= cb_until && n - c >= KLPM_FAST_CTA_MIN) {
                if (lane == 0) {
                    s_bio.cur = cur; s_bio.head = head; s_bio.c = c; s_bio.cyc = cyc; s_bio.root = root; s_bio.B = 0;
                    s_job.type = FAST_JOB_BATCH;
                }
                __syncwarp();
                const long long t_cta = clock64();
                ++n_cta_try;
                named_bar(1, KLPM_FAST_THREADS);
                fast_batch_job<G>(A, R, &s_bio, sr, sr + 1024, sr + 2048, reinterpret_cast<int32_t*>(sh), s_scan, nwords);
                const int32_t Bc = s_bio.B;
                const long long cy_this = clock64() - t_cta;
                cy_cta += cy_this;
                if (Bc > 0) {
                    ++n_cta_ok; dec_cta += Bc;
                    const int32_t consumed = s_bio.consumed, hmax = s_bio.hmax;
                    c += Bc;
                    one_next = s_bio.hard != 0;
                    if (A.policy == KLPM_POLICY_KLPM) cyc = (cyc + Bc) % A.k;
                    if (consumed) { cur += consumed; window(cur & ~31, &wk, &ws); window((cur & ~31) + 32, &nk, &ns); }
                    if (hmax >= 0) { head = hmax; advance_head(); }
                    else if (head < n && ((bm_ld(s_done, head >> 5, gdone) >> (head & 31)) & 1u)) advance_head();
                    // did it pay?  its cycles per decision against what the warp-wide steps have cost per decision so far
                    const long long warp_cpd = dec_warp >= 256 ? cy_warp / dec_warp : 100;
                    if (cy_this <= (long long)Bc * warp_cpd) { cb_back = 8; cb_fail = 0; continue; }
                    // committed, but too short to have paid for the attempt: warp-wide steps for a while, as after a failure
                    cb_wait = cb_back;
                    cb_back = cb_back < KLPM_FAST_CB_MAX ? cb_back * 2 : KLPM_FAST_CB_MAX;
                    calm = 0;
                    continue;
                }
                // too few decisions before one that needs the one-at-a-time path: the next attempt waits until that one has
                // been made (and longer when attempts keep failing: such decisions come in runs)
                cb_until = c + s_bio.Braw + 1 + (cb_fail > 0 ? (8 << cb_fail) : 0);
                if (cb_fail < KLPM_FAST_FAIL_CAP) ++cb_fail;
            }
            --cb_wait;
            if (!one_next && vb_wait <= 0) {
                const int32_t c_was = c;
                const long long t_w = clock64();
                const bool took = try_batch();
                cy_warp += clock64() - t_w;
                if (took) { ++n_warp_ok; dec_warp += c - c_was; vb_back = 1; calm = c - c_was == 32 ? calm + 1 : 0; one_next = tb_cut; continue; }
                calm = 0;
                vb_wait = vb_back;
                vb_back = vb_back < 64 ? vb_back * 2 : 64;
            }
            if (!one_next) --vb_wait;
            one_next = false;
            ++dec_one;
            const bool fcfs_turn = A.policy == KLPM_POLICY_FCFS || (A.policy == KLPM_POLICY_KLPM && cyc == 0);
            if (++cyc == A.k) cyc = 0;
            int32_t j;
            bool in_tour;                                   // the pick's key is in the tournament (it changed after the sort)
            if (fcfs_turn) {
                j = head;
                in_tour = (bm_ld(R.skip, j >> 5, gbits) >> (j & 31)) & 1u;
            } else {
                unsigned long long ek = 0;                  // next entry of the list that still counts
                int32_t es = -1;
                while (cur < n) {                           // (a window's 32 entries are examined at once: stale entries come in runs)
                    const int32_t wbase = cur & ~31;
                    const bool usable = lane >= (cur & 31) && (long long)wbase + lane < n && !((bm_ld(R.skip, ws >> 5, gbits) >> (ws & 31)) & 1u);
                    const unsigned bal = __ballot_sync(FULL_MASK, usable);
                    if (bal) {
                        const int src = __ffs(bal) - 1;
                        cur = wbase + src;
                        const long long kk = __shfl_sync(FULL_MASK, wk, src);
                        es = __shfl_sync(FULL_MASK, ws, src);
                        ek = ~((unsigned long long)kk ^ 0x8000000000000000ULL);
                        break;
                    }
                    cur = wbase + 32; wk = nk; ws = ns; window(cur + 32, &nk, &ns);
                }
                if (cur > n) cur = n;
                if (root > ek) {
                    const unsigned rk = 0xffffffffu - (unsigned)(root & 0xffffffffULL);
                    j = A.pinv ? __ldg(A.pinv + rk) : (int32_t)rk;
                    in_tour = true;
                } else {
                    j = es;
                    in_tour = false;
                    advance_cur();
                }
            }
            if (j < 0 || j >= n || ((bm_ld(s_done, j >> 5, gdone) >> (j & 31)) & 1u)) { if (lane == 0) set_status(A.st, RT_ERR_LIMIT, 107); failed = true; break; }   // cannot happen
            mark_done(j);
            if (in_tour) {                                  // its leaf block's largest changed key, without it
                const int32_t b = j >> A.lb_shift;
                unsigned long long kk;
                if (!G && A.lb_shift == 5) {                // 32-slot blocks, bitmaps in shared memory: one word of each
                    const unsigned w = R.skip[b] & ~s_done[b];
                    kk = warp_max64r(((w >> lane) & 1u) ? __ldcg(A.key + ((long long)b << 5) + lane) : 0ULL);
                } else {
                    kk = changed_block_max(A, R, b, lane);
                }
                root = tour_set(R, b, kk, lane);
            }
            if (j == head) advance_head();
            if ((bm_ld(R.gb, j >> 5, gbits) >> (j & 31)) & 1u) {
                careful(j, false, ld_dyn(A.dyn + j), ld_stat(A.stat + j));
            } else {
                if (lane == 0) A.order[c] = j;
                ++c;
            }
        }
        if (lane == 0) {
            long long* cn = A.post->counters;
            cn[8] = n_cta_try; cn[9] = n_cta_ok; cn[10] = dec_cta; cn[11] = n_warp_ok; cn[12] = dec_warp; cn[13] = dec_one;
            cn[14] = cy_cta; cn[15] = cy_warp;
        }
    } else if (lane == 0) {
        A.post->c0 = n;                                     // list mode never began: nothing is left to charge
        A.post->now0 = now;
        for (int i = 8; i < 16; ++i) A.post->counters[i] = 0;
    }
    __syncwarp();
    if (lane == 0) {
        long long* cn = A.post->counters;
        cn[0] = n_careful; cn[1] = n_cta_dissolve; cn[2] = n_scan; cn[3] = s_memcur - (A.lru ? 2 * n : n); cn[4] = n_evict;
        cn[5] = cy_tree; cn[6] = cy_scan; cn[7] = cy_dissolve;
    }
    if (A.lru && lane == 0) {                               // the tree's counters go back (a status recorded meanwhile stays)
        TreeState out = s_st;
        out.status = *reinterpret_cast<const volatile int*>(&A.st->status);
        out.detail = *reinterpret_cast<const volatile int*>(&A.st->detail);
        *A.st = out;
    }
    if (lane == 0) s_job.type = FAST_JOB_EXIT;
    __syncwarp();
    named_bar(1, KLPM_FAST_THREADS);
}

// The charge pass after the loop: the decisions made in list mode, c0 .. n-1, are in `order` as slots.  Nobody waited
// for an arrival there, so completion times are the time list mode began plus a running sum of the costs
// (Definition 2 with R_prev >= t_j).  Three small kernels: per decision its uncached tokens and cost (and the query
// index put in `order`), a scan of the per-block sums, and the completion times and TTFTs.
#define KLPM_CHARGE_THREADS 256
// `ipt` consecutive decisions per thread: at most 1,024 blocks whatever the queue's length.
__global__ void __launch_bounds__(KLPM_CHARGE_THREADS)
charge_cost_kernel(FastArgs A, long long* cost, long long* bsum, int32_t ipt) {
    __shared__ long long s_w[KLPM_CHARGE_THREADS / 32];
    const long long i0 = ((long long)blockIdx.x * blockDim.x + threadIdx.x) * ipt;
    long long x = 0;
    for (int32_t u = 0; u < ipt; ++u) {
        const long long i = i0 + u, c = A.post->c0 + i;
        if (c < A.n) {
            const int32_t slot = A.order[c];
            const int4 s = __ldg(reinterpret_cast<const int4*>(A.stat + slot));     // arrival, length, query index
            const int32_t len = s.z, ord = s.w, unc = len - A.dyn[slot].m;
            const long long y = (A.c_den + A.c_num * (long long)len) * (long long)unc;
            A.order[c] = ord;
            A.uncached[ord] = unc;
            cost[i] = y;
            x += y;
        }
    }
#pragma unroll
    for (int d = 16; d > 0; d >>= 1) x += __shfl_down_sync(FULL_MASK, x, d);
    if ((threadIdx.x & 31) == 0) s_w[threadIdx.x >> 5] = x;
    __syncthreads();
    if (threadIdx.x == 0) {
        long long sum = 0;
        for (int w = 0; w < KLPM_CHARGE_THREADS / 32; ++w) sum += s_w[w];
        bsum[blockIdx.x] = sum;
    }
}
// bsum[b] <- time at which block b's first decision starts (at most 1,024 blocks)
__global__ void __launch_bounds__(1024)
charge_scan_kernel(FastArgs A, long long* bsum, int32_t nblocks) {
    __shared__ long long s[1024];
    const int u = threadIdx.x;
    const long long v = u < nblocks ? bsum[u] : 0;
    s[u] = v;
    __syncthreads();
    for (int d = 1; d < 1024; d <<= 1) {
        const long long o = u >= d ? s[u - d] : 0;
        __syncthreads();
        s[u] += o;
        __syncthreads();
    }
    if (u < nblocks) bsum[u] = A.post->now0 + s[u] - v;
}
__global__ void __launch_bounds__(KLPM_CHARGE_THREADS)
charge_apply_kernel(FastArgs A, const long long* cost, const long long* bsum, int32_t ipt) {
    __shared__ long long s_w[KLPM_CHARGE_THREADS / 32];
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    const long long i0 = ((long long)blockIdx.x * blockDim.x + threadIdx.x) * ipt;
    long long mine = 0;                                     // cost of this thread's decisions
    for (int32_t u = 0; u < ipt; ++u) { const long long c = A.post->c0 + i0 + u; if (c < A.n) mine += cost[i0 + u]; }
    long long x = mine;
#pragma unroll
    for (int d = 1; d < 32; d <<= 1) { const long long o = __shfl_up_sync(FULL_MASK, x, d); if (lane >= d) x += o; }
    if (lane == 31) s_w[warp] = x;
    __syncthreads();
    long long run = bsum[blockIdx.x] + x - mine;            // time at which this thread's first decision starts
    for (int w = 0; w < warp; ++w) run += s_w[w];
    for (int32_t u = 0; u < ipt; ++u) {
        const long long i = i0 + u, c = A.post->c0 + i;
        if (c < A.n) {
            const int32_t ord = A.order[c];
            run += cost[i];
            A.ttft[ord] = run - A.arrival[ord];
            if (A.completion) A.completion[ord] = run;
        }
    }
}

// ------------------------------------------------------------------------------------------------
// bulk insertion of many prompts into a tree without a budget.  The set of node boundaries a radix tree
// ends up with does not depend on the order in which prompts are stored, so prompts are inserted in
// rounds: every pending prompt is walked from the root (read-only), then at most one prompt per edge
// cuts that edge, and prompts that end at a node boundary add their leaves concurrently (the hash
// table's compare-and-swap on the key decides between prompts that want the same child).
// ------------------------------------------------------------------------------------------------
struct BulkArgs {
    const int32_t* tok; const int64_t* off;
    const int32_t* pend_in; int32_t* pend_out; unsigned int* n_out;   // walk: prompts to walk -> prompts not fully stored yet
    int32_t* pend_next; unsigned int* n_next;                          // apply: prompts that have to try again next round
    unsigned int* n_walk;                                              // walk: work counter
    int32_t* claim;                    // per node: lowest prompt index that wants to cut its edge
    int32_t* pm; int32_t* pnode; int32_t* poff;   // per prompt: where its walk ended
};

__global__ void __launch_bounds__(256)
bulk_walk_kernel(TreeDev T, BulkArgs A, unsigned n_pending) {
    const int lane = threadIdx.x & 31;
    for (;;) {                                              // prompts are handed out by a counter: their lengths differ widely
        unsigned p = 0;
        if (lane == 0) p = atomicAdd(A.n_walk, 1u);
        p = __shfl_sync(FULL_MASK, p, 0);
        if (p >= n_pending) return;
        const int32_t i = __ldg(A.pend_in + p);
        const int64_t lo = __ldg(A.off + i);
        const int32_t len = (int32_t)(__ldg(A.off + i + 1) - lo);
        // the tree has no budget, so the walk streams along contiguous pool runs (as the batched match does)
        int32_t node, off;
        const int32_t m = walk_chain(T, A.tok + lo, len, true, &node, &off);
        const bool full = node == 0 || off == __ldg(T.span_len + node);     // ends on a node boundary (or at the root)
        if (lane == 0 && !(m == len && full)) {
            A.pm[i] = m; A.pnode[i] = node; A.poff[i] = full ? -1 : off;
            if (!full) atomicMin(&A.claim[node], i);
            A.pend_out[atomicAdd(A.n_out, 1u)] = i;
        }
    }
}

// First round when a batched match of the prompts against the tree as it still is has left its records (MatchState):
// the node where each match ended is looked up from the position (end_node[] along the run), then what
// bulk_walk_kernel does after its walk.  One lane per prompt, 32 prompts of the list per warp at a time; the search
// along a run for a match that ended inside an edge is the whole warp's, one prompt after the other; the list of
// pending prompts grows by one addition per warp.
__global__ void __launch_bounds__(256)
bulk_from_state_kernel(TreeDev T, BulkArgs A, const MatchState* __restrict__ state, unsigned long long tag, unsigned n_pending) {
    const int lane = threadIdx.x & 31;
    const unsigned nwarps = (gridDim.x * blockDim.x) >> 5;
    const EndIndex X = end_index(T);
    for (unsigned long long p0 = (unsigned long long)((blockIdx.x * blockDim.x + threadIdx.x) >> 5) * 32ULL; p0 < n_pending;
         p0 += (unsigned long long)nwarps * 32ULL) {
        const unsigned long long p = p0 + lane;
        int32_t i = -1;
        if (p < n_pending) i = A.pend_in[p];                 // < 0: a replay that stopped early, not processed
        bool act = i >= 0, inside = false;
        int32_t len = 0, m = 0, node = 0, off = -1;          // off < 0: the match ends on a node boundary (or at the root)
        long long pos = -1, cend = 0;
        if (act) {
            len = (int32_t)(__ldg(A.off + i + 1) - __ldg(A.off + i));
            const int4* src = reinterpret_cast<const int4*>(state + i);
            const int4 a = __ldcg(src), b = __ldcg(src + 1);
            pos = (long long)(((unsigned long long)(unsigned)a.y << 32) | (unsigned)a.x);
            cend = (long long)(((unsigned long long)(unsigned)a.w << 32) | (unsigned)a.z);
            m = b.x;
            const unsigned long long got = ((unsigned long long)(unsigned)b.w << 32) | (unsigned)b.z;
            if (got != tag || m < 0 || m > len || pos < -1 || pos >= T.max_pool || cend < 0 || cend > T.max_pool) {
                set_status(T.st, RT_ERR_INVALID, 110);      // not a record of that match: the prompt is left out
                act = false;
            } else if (pos >= 0) {
                node = node_ending_at(X, pos, *reinterpret_cast<const volatile long long*>(&T.st->n_nodes));
                inside = node < 0;
            }
        }
        unsigned im = __ballot_sync(FULL_MASK, inside);
        while (im) {
            const int src = __ffs(im) - 1; im &= im - 1;
            const int32_t r = node_after(X, __shfl_sync(FULL_MASK, pos, src), __shfl_sync(FULL_MASK, cend, src));
            if (lane == src) {
                if (r < 0) { set_status(T.st, RT_ERR_LIMIT, 111); act = false; }      // cannot happen
                else { node = r; off = m - __ldg(T.depth_start + r); }
            }
        }
        const bool pend = act && !(m == len && off < 0);
        if (pend) {
            A.pm[i] = m; A.pnode[i] = node; A.poff[i] = off;
            if (off >= 0) atomicMin(&A.claim[node], i);
        }
        const unsigned pm = __ballot_sync(FULL_MASK, pend);
        if (pm) {
            const int lead = __ffs(pm) - 1;
            unsigned base = 0;
            if (lane == lead) base = atomicAdd(A.n_out, (unsigned)__popc(pm));
            base = __shfl_sync(FULL_MASK, base, lead);
            if (pend) A.pend_out[base + __popc(pm & ((1u << lane) - 1u))] = i;
        }
    }
}

// What the apply step does for 32 pending prompts of the list (one per lane, from number p0 on): cut the edge the
// match ends in if the prompt holds the claim, add its leaf if it wins the child's table slot, or put the prompt on
// the list for the next round; then the warp copies the new leaves' tokens, one leaf after the other.  New nodes are
// numbered and pool space is taken with one addition per warp.  Tree fields are read through L2 (__ldcg): inside the
// kernel that runs all later rounds, another SM may have written them a moment ago.
__device__ __forceinline__ void bulk_apply_warp(const TreeDev& T, const BulkArgs& A, unsigned long long p0, unsigned n_apply, int lane,
                                                unsigned long long* s_live_nodes, unsigned long long* s_live_tokens) {
    TreeState* S = T.st;
    const unsigned lt = (1u << lane) - 1u;
    const bool act = p0 + lane < n_apply;
    int32_t i = 0, len = 0, m = 0, node = 0, off = -1;
    const int32_t* x = A.tok;
    if (act) {
        i = __ldcg(A.pend_out + p0 + lane);
        const int64_t lo = __ldg(A.off + i);
        len = (int32_t)(__ldg(A.off + i + 1) - lo);
        x = A.tok + lo;
        m = __ldcg(A.pm + i); node = __ldcg(A.pnode + i); off = __ldcg(A.poff + i);
    }
    const int32_t unc = len - m;
    bool go = act, retry = false;
    int32_t end = node;
    // ---- the match ends inside node's edge: cut it, unless another prompt cuts this edge in this round
    bool cut = act && off >= 0;
    if (cut && __ldcg(A.claim + node) != i) { cut = false; go = false; retry = true; }
    const unsigned cm = __ballot_sync(FULL_MASK, cut);
    if (cm) {
        const int lead = __ffs(cm) - 1;
        unsigned long long base = 0;
        if (lane == lead) base = atomicAdd((unsigned long long*)&S->n_nodes, (unsigned long long)__popc(cm));
        base = __shfl_sync(FULL_MASK, base, lead);
        if (cut) {
            const long long u = (long long)base + __popc(cm & lt);
            A.claim[node] = 0x7fffffff;
            if (u >= T.max_nodes) { set_status(S, RT_ERR_CAPACITY); go = false; }
            else {
                atomicAdd(s_live_nodes, 1ULL);
                const int32_t par = __ldcg(T.parent + node), ds = __ldcg(T.depth_start + node), sl = __ldcg(T.span_len + node);
                const int64_t so = __ldcg(T.span_off + node);
                const int32_t t_up = __ldcg(T.pool + so), t_low = __ldcg(T.pool + so + off);
                T.parent[u] = par; T.depth_start[u] = ds; T.span_off[u] = so; T.span_len[u] = off;
                T.nchild[u] = 1; T.dead[u] = 0; T.last_access[u] = 0;
                T.first_tok[u] = t_up; T.first_tok[node] = t_low;
                long long slot = table_find(T, par, t_up);
                int64_t chain_end = so + sl;
                if (slot >= 0) { T.table[slot].child = (int32_t)u; T.table[slot].span_len = off; chain_end = __ldcg(&T.table[slot].chain_end); }
                else set_status(S, RT_ERR_LIMIT, 104);
                T.end_node[so + off - 1] = (int32_t)u;
                T.span_off[node] = so + off; T.span_len[node] = sl - off; T.depth_start[node] = ds + off;
                T.parent[node] = (int32_t)u;
                end = (int32_t)u;
                // (u, first token of the lower part) -> node : nobody else can want this key
                unsigned long long key = make_key(end, t_low);
                unsigned long long sl2 = hash_key(key) & T.table_mask;
                for (unsigned long long pr = 0; pr <= T.table_mask; ++pr) {
                    if (atomicCAS(&T.table[sl2].key, 0ULL, key) == 0ULL) {
                        T.table[sl2].child = node; T.table[sl2].span_len = sl - off; T.table[sl2].span_off = so + off;
                        T.table[sl2].chain_end = chain_end;
                        break;
                    }
                    sl2 = (sl2 + 1) & T.table_mask;
                }
            }
        }
    }
    // ---- the leaf: whoever puts the child's key into the table adds it
    long long won = -1;
    if (go && unc > 0) {
        unsigned long long key = make_key(end, __ldg(x + m));
        unsigned long long sl2 = hash_key(key) & T.table_mask;
        for (unsigned long long pr = 0; pr <= T.table_mask; ++pr) {
            unsigned long long old = atomicCAS(&T.table[sl2].key, 0ULL, key);
            if (old == 0ULL) { won = (long long)sl2; break; }
            if (old == key) { retry = true; break; }       // another prompt added that child (in this round, or it lost to it before)
            sl2 = (sl2 + 1) & T.table_mask;
        }
    }
    int64_t dst = -1;
    const unsigned wm = __ballot_sync(FULL_MASK, won >= 0);
    if (wm) {
        const long long need = won >= 0 ? (long long)unc + 6 : 0;
        long long inc = need;
#pragma unroll
        for (int d = 1; d < 32; d <<= 1) { const long long o = __shfl_up_sync(FULL_MASK, inc, d); if (lane >= d) inc += o; }
        const long long tot = __shfl_sync(FULL_MASK, inc, 31);
        unsigned long long nb = 0, pb = 0;
        if (lane == 0) {
            nb = atomicAdd((unsigned long long*)&S->n_nodes, (unsigned long long)__popc(wm));
            pb = atomicAdd((unsigned long long*)&S->pool_used, (unsigned long long)tot);
        }
        nb = __shfl_sync(FULL_MASK, nb, 0); pb = __shfl_sync(FULL_MASK, pb, 0);
        if (won >= 0) {
            const long long leaf = (long long)nb + __popc(wm & lt);
            const long long raw = (long long)pb + inc - need;
            const long long po = ((raw + 3) & ~3LL) + (m & 3);                  // span_off = depth_start (mod 4)
            if (leaf >= T.max_nodes || raw + unc + 6 > T.max_pool) {
                set_status(S, RT_ERR_CAPACITY);
                T.table[won].child = -1; T.table[won].span_len = 0; T.table[won].span_off = 0; T.table[won].chain_end = 0;
            } else {
                T.parent[leaf] = end; T.depth_start[leaf] = m; T.span_off[leaf] = po; T.span_len[leaf] = unc;
                T.nchild[leaf] = 0; T.dead[leaf] = 0; T.last_access[leaf] = 0;
                T.first_tok[leaf] = __ldg(x + m);
                T.table[won].child = (int32_t)leaf; T.table[won].span_len = unc; T.table[won].span_off = po;
                T.table[won].chain_end = po + unc;
                T.end_node[po + unc - 1] = (int32_t)leaf;
                atomicAdd(&T.nchild[end], 1);
                atomicAdd(s_live_tokens, (unsigned long long)unc);
                atomicAdd(s_live_nodes, 1ULL);
                dst = po;
            }
        }
    }
    const unsigned rm = __ballot_sync(FULL_MASK, retry);
    if (rm) {
        const int lead = __ffs(rm) - 1;
        unsigned base = 0;
        if (lane == lead) base = atomicAdd(A.n_next, (unsigned)__popc(rm));
        base = __shfl_sync(FULL_MASK, base, lead);
        if (retry) A.pend_next[base + __popc(rm & lt)] = i;
    }
    // ---- the new leaves' tokens
    unsigned dm = __ballot_sync(FULL_MASK, dst >= 0);
    while (dm) {
        const int src = __ffs(dm) - 1; dm &= dm - 1;
        const int64_t d = __shfl_sync(FULL_MASK, dst, src);
        const int32_t* xs = reinterpret_cast<const int32_t*>(__shfl_sync(FULL_MASK, (unsigned long long)(x + m), src));
        const int32_t cnt = __shfl_sync(FULL_MASK, unc, src);
        for (int32_t t0 = 0; t0 < cnt; t0 += 128) {
            int32_t v[4];
#pragma unroll
            for (int r = 0; r < 4; ++r) { const int32_t t = t0 + r * 32 + lane; v[r] = t < cnt ? __ldg(xs + t) : 0; }
#pragma unroll
            for (int r = 0; r < 4; ++r) { const int32_t t = t0 + r * 32 + lane; if (t < cnt) T.pool[d + t] = v[r]; }
        }
    }
}

__global__ void __launch_bounds__(256)
bulk_apply_kernel(TreeDev T, BulkArgs A) {
    // live nodes and live tokens are statistics only: summed per CTA here, added to the tree's counters once at the end
    __shared__ unsigned long long s_live_nodes, s_live_tokens;
    if (threadIdx.x == 0) { s_live_nodes = 0ULL; s_live_tokens = 0ULL; }
    __syncthreads();
    const unsigned n_pending = *A.n_out;
    const int lane = threadIdx.x & 31;
    const unsigned nwarps = (gridDim.x * blockDim.x) >> 5;
    for (unsigned long long p0 = (unsigned long long)((blockIdx.x * blockDim.x + threadIdx.x) >> 5) * 32ULL; p0 < n_pending;
         p0 += (unsigned long long)nwarps * 32ULL)
        bulk_apply_warp(T, A, p0, n_pending, lane, &s_live_nodes, &s_live_tokens);
    __syncthreads();
    if (threadIdx.x == 0) {
        if (s_live_nodes) atomicAdd((unsigned long long*)&T.st->live_nodes, s_live_nodes);
        if (s_live_tokens) atomicAdd((unsigned long long*)&T.st->tokens_live, s_live_tokens);
    }
}

// Every round after the first, in one cooperative kernel (no trip to the host between rounds).  A round = bring the
// pending prompts' positions up to date, grid barrier, apply, grid barrier.  A prompt is pending because it lost a
// cut to another prompt -- then the depth where its match ends has not moved, only the nodes around it have, and a
// walk up from the node it knew finds the node that holds that depth now -- or because another prompt added the
// child it wanted -- then it walks on from the node boundary it had reached, into that child (hop by hop, read
// through L2: the tokens may have been written by another SM a moment ago).  Counters alternate between rounds so
// that none is reset while somebody may still read it.  The barrier is bounded in time; when it gives up the status
// word says RT_ERR_LIMIT and every CTA returns.
struct BulkSync {
    unsigned int count, gen, abort, go;      // the barrier; whether another round follows
    unsigned int cnt_w[2], cnt_a[2];         // list lengths: positions brought up to date -> pend_b; retries -> pend_a
    unsigned int n_walk;                     // work counter of the first round's walk
    unsigned int pad[3];
};

// All threads call it.  `last` runs in one thread of the CTA that arrives last, before anybody is released.
template <typename F>
__device__ bool bulk_barrier(BulkSync* g, TreeState* st, long long limit_ns, F last) {
    __shared__ int s_ok;
    __threadfence();
    __syncthreads();
    if (threadIdx.x == 0) {
        int ok = 1;
        const unsigned gen = *(volatile unsigned*)&g->gen;
        if (atomicAdd(&g->count, 1u) + 1u == gridDim.x) {
            last();
            g->count = 0;
            __threadfence();
            atomicAdd(&g->gen, 1u);
        } else {
            unsigned long long spins = 0, t0 = 0;
            while (*(volatile unsigned*)&g->gen == gen) {
                if (*(volatile unsigned*)&g->abort) { ok = 0; break; }
                if ((++spins & 1023ULL) == 0 || limit_ns == 0) {
                    unsigned long long now;
                    asm volatile("mov.u64 %0, %globaltimer;" : "=l"(now));
                    if (t0 == 0) t0 = now;
                    if (limit_ns == 0 || now - t0 > (unsigned long long)limit_ns || spins > (1ULL << 40)) {
                        set_status(st, RT_ERR_LIMIT, 112); atomicExch(&g->abort, 1u); ok = 0; break;
                    }
                }
            }
        }
        if (*(volatile unsigned*)&g->abort) ok = 0;
        __threadfence();
        s_ok = ok;
    }
    __syncthreads();
    const bool ok = s_ok != 0;
    __syncthreads();
    return ok;
}

__global__ void __launch_bounds__(256)
bulk_rounds_kernel(TreeDev T, BulkArgs A, BulkSync* g, long long n_total, const int32_t* n_total_dev, long long limit_ns) {
    __shared__ unsigned long long s_live_nodes, s_live_tokens;
    if (threadIdx.x == 0) { s_live_nodes = 0ULL; s_live_tokens = 0ULL; }
    __syncthreads();
    const int lane = threadIdx.x & 31;
    const unsigned nwarps = (gridDim.x * blockDim.x) >> 5, warp0 = (blockIdx.x * blockDim.x + threadIdx.x) >> 5;
    TreeState* S = T.st;
    unsigned count = __ldcg(&g->cnt_a[0]);                 // left pending by the first round (its kernels have completed)
    for (unsigned r = 1; count > 0; ++r) {
        const unsigned par = r & 1u;
        BulkArgs R = A;
        R.pend_in = A.pend_next; R.n_out = &g->cnt_w[par]; R.n_next = &g->cnt_a[par];
        // ---- positions of the pending prompts in the tree as it is now
        for (unsigned p = warp0; p < count; p += nwarps) {
            const int32_t i = __ldcg(R.pend_in + p);
            const int64_t lo = __ldg(A.off + i);
            const int32_t len = (int32_t)(__ldg(A.off + i + 1) - lo);
            int32_t m = __ldcg(A.pm + i), node = __ldcg(A.pnode + i), off = __ldcg(A.poff + i);
            bool full = true;
            if (off >= 0) {                                 // lost a cut: the depth m lies in `node` or in a node cut off above it
                int32_t a = node, ds = __ldcg(T.depth_start + a);
                while (a != 0 && m <= ds) { a = __ldcg(T.parent + a); ds = __ldcg(T.depth_start + a); }
                node = a; off = m - ds;
                full = a == 0 || off == __ldcg(T.span_len + a);
            }
            if (full) {                                     // on a node boundary: walk on into the child that may be there now
                const Term t = walk<false>(T, A.tok + lo, len, node, m);
                if (t.m > m) { m = t.m; node = t.node; off = t.off; full = t.full != 0; }
            }
            if (lane == 0 && !(m == len && full)) {
                A.pm[i] = m; A.pnode[i] = node; A.poff[i] = full ? -1 : off;
                if (!full) atomicMin(&A.claim[node], i);
                R.pend_out[atomicAdd(R.n_out, 1u)] = i;
            }
        }
        if (!bulk_barrier(g, S, limit_ns, [] {})) break;
        // ---- cuts and leaves
        const unsigned n_apply = __ldcg(R.n_out);
        if (blockIdx.x == 0 && threadIdx.x == 0) { g->cnt_w[par ^ 1u] = 0u; g->cnt_a[par ^ 1u] = 0u; }     // the next round's
        for (unsigned long long p0 = (unsigned long long)warp0 * 32ULL; p0 < n_apply; p0 += (unsigned long long)nwarps * 32ULL)
            bulk_apply_warp(T, R, p0, n_apply, lane, &s_live_nodes, &s_live_tokens);
        if (!bulk_barrier(g, S, limit_ns, [&] {
                const bool stop = *(volatile int*)&S->status != 0 || r > 100000000u;
                g->go = stop ? 0u : *(volatile unsigned*)&g->cnt_a[par];
            })) break;
        count = __ldcg(&g->go);
    }
    __syncthreads();
    if (threadIdx.x == 0) {
        if (s_live_nodes) atomicAdd((unsigned long long*)&S->live_nodes, s_live_nodes);
        if (s_live_tokens) atomicAdd((unsigned long long*)&S->tokens_live, s_live_tokens);
        if (blockIdx.x == 0) {                              // the logical clock advances by one per stored prompt
            if (n_total_dev) n_total = *n_total_dev;
            if (S->clock + n_total + 1 >= T.max_clock) set_status(S, RT_ERR_CAPACITY);
            else S->clock += n_total;
        }
    }
}

__global__ void bulk_iota_kernel(int32_t* p, int32_t n) {
    int32_t i = blockIdx.x * blockDim.x + threadIdx.x;
    if (i < n) p[i] = i;
}
__global__ void bulk_fill_kernel(int32_t* p, long long n, int32_t v) {
    long long i = (long long)blockIdx.x * blockDim.x + threadIdx.x;
    if (i < n) p[i] = v;
}
// ------------------------------------------------------------------------------------------------
// Many independent small queues under the last-prompt cache (Definition 2 as printed; Section 2.1: only the
// previously processed prompt is cached).  This is the model the paper's worked example and Theorem 2 speak
// about, and a Monte-Carlo over random arrival orders (Definition 3) is thousands of such queues: one warp runs
// one queue from start to finish, so the schedule loop itself is what is data-parallel here.
// Per decision the warp looks at every prompt of its queue, 32 at a time: who has arrived, who is oldest, and --
// for a longest-match pick -- overlap(x_i, last processed prompt), computed by the whole warp for the prompts
// whose first token agrees with it.  The processed flags live in shared memory (one bit per prompt).
// ------------------------------------------------------------------------------------------------
#define KLPM_LAST_ONLY_WARPS 4
struct LastOnlyArgs {
    const int32_t* tok; const int64_t* off; const int64_t* arrival; const int64_t* prio; const int32_t* qoff;
    int32_t n_queues;
    int32_t policy, k;
    long long c_num, c_den, start_tick;
    int32_t* order; int32_t* uncached; int64_t* ttft; int64_t* completion; int32_t* n_skipped;
};

__global__ void __launch_bounds__(32 * KLPM_LAST_ONLY_WARPS)
last_only_batch_kernel(LastOnlyArgs A) {
    __shared__ unsigned s_done[KLPM_LAST_ONLY_WARPS][KLPM_LAST_ONLY_MAX_QUEUE / 32];
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    const long long r = (long long)blockIdx.x * KLPM_LAST_ONLY_WARPS + warp;
    if (r >= A.n_queues) return;
    const int32_t q0 = __ldg(A.qoff + r), n = __ldg(A.qoff + r + 1) - q0;
    if (n <= 0) return;
    if (n > KLPM_LAST_ONLY_MAX_QUEUE) {                       // too long for this entry point: left untouched, counted
        if (lane == 0 && A.n_skipped) atomicAdd(A.n_skipped, 1);
        return;
    }
    unsigned* done = s_done[warp];
    for (int32_t w = lane; w < KLPM_LAST_ONLY_MAX_QUEUE / 32; w += 32) done[w] = 0u;
    __syncwarp();
    const long long INF = 0x7fffffffffffffffLL;
    long long now = A.start_tick;
    int32_t last = -1, last_len = 0;                          // the cached prompt (global index) and its length
    const int32_t* last_x = nullptr;
    for (int32_t c = 0; c < n; ++c) {
        // ---- who is waiting; if nobody, idle until the next arrival
        bool any = false;
        long long tmin = INF;
        for (int32_t base = 0; base < n; base += 32) {
            const int32_t i = base + lane;
            if (i < n && !((done[i >> 5] >> (i & 31)) & 1u)) {
                const long long t = __ldg(A.arrival + q0 + i);
                any = any || t <= now;
                tmin = t < tmin ? t : tmin;
            }
        }
        any = __any_sync(FULL_MASK, any);
        if (!any) {
#pragma unroll
            for (int d = 16; d > 0; d >>= 1) { const long long o = __shfl_xor_sync(FULL_MASK, tmin, d); tmin = o < tmin ? o : tmin; }
            now = tmin;
        }
        const bool fcfs_turn = A.policy == KLPM_POLICY_FCFS || (A.policy == KLPM_POLICY_KLPM && (c % A.k) == 0);
        // ---- the pick: best of (score desc, priority asc, arrival asc, index asc); score = 0 on an oldest-first turn,
        //      and the priority plays no part in it
        int32_t b_idx = -1, b_score = 0;
        long long b_prio = 0, b_t = 0;
        for (int32_t base = 0; base < n; base += 32) {
            const int32_t i = base + lane;
            bool waiting = false;
            long long t = 0, pr = 0;
            int32_t len = 0;
            const int32_t* x = nullptr;
            if (i < n && !((done[i >> 5] >> (i & 31)) & 1u)) {
                t = __ldg(A.arrival + q0 + i);
                waiting = t <= now;
            }
            int32_t score = 0;
            if (!fcfs_turn) {
                bool cmp = false;
                if (waiting) {
                    const int64_t lo = __ldg(A.off + q0 + i);
                    len = (int32_t)(__ldg(A.off + q0 + i + 1) - lo);
                    x = A.tok + lo;
                    if (A.prio) pr = __ldg(A.prio + q0 + i);
                    cmp = last >= 0 && len > 0 && last_len > 0 && __ldg(x) == __ldg(last_x);
                }
                unsigned cm = __ballot_sync(FULL_MASK, cmp);
                while (cm) {                                  // overlap(x_i, last): the whole warp compares one prompt at a time
                    const int src = __ffs(cm) - 1; cm &= cm - 1;
                    const int32_t* xs = (const int32_t*)__shfl_sync(FULL_MASK, (unsigned long long)x, src);
                    const int32_t ls = __shfl_sync(FULL_MASK, len, src);
                    const int32_t e = first_mismatch<true, 1>(xs, last_x, ls < last_len ? ls : last_len);
                    if (lane == src) score = e;
                }
            }
            if (waiting) {
                bool wins = b_idx < 0 || score > b_score;
                if (!wins && score == b_score) {
                    if (pr != b_prio) wins = pr < b_prio;
                    else wins = t < b_t || (t == b_t && i < b_idx);
                }
                if (wins) { b_idx = i; b_score = score; b_prio = pr; b_t = t; }
            }
        }
#pragma unroll
        for (int d = 16; d > 0; d >>= 1) {
            const int32_t o_idx = __shfl_xor_sync(FULL_MASK, b_idx, d), o_score = __shfl_xor_sync(FULL_MASK, b_score, d);
            const long long o_prio = __shfl_xor_sync(FULL_MASK, b_prio, d), o_t = __shfl_xor_sync(FULL_MASK, b_t, d);
            bool wins = o_idx >= 0 && (b_idx < 0 || o_score > b_score);
            if (!wins && o_idx >= 0 && b_idx >= 0 && o_score == b_score) {
                if (o_prio != b_prio) wins = o_prio < b_prio;
                else wins = o_t < b_t || (o_t == b_t && o_idx < b_idx);
            }
            if (wins) { b_idx = o_idx; b_score = o_score; b_prio = o_prio; b_t = o_t; }
        }
        const int32_t j = b_idx;                               // somebody is waiting, so j >= 0
        if (j < 0) return;
        // ---- charge by Definition 2 against the cached prompt, then x_j is the cached prompt
        const int64_t lo = __ldg(A.off + q0 + j);
        const int32_t len = (int32_t)(__ldg(A.off + q0 + j + 1) - lo);
        const int32_t* x = A.tok + lo;
        int32_t m = 0;
        if (last >= 0) m = first_mismatch<true, 1>(x, last_x, len < last_len ? len : last_len);
        const int32_t unc = len - m;
        const long long tj = __ldg(A.arrival + q0 + j);
        const long long begin = now > tj ? now : tj;
        const long long R = begin + (A.c_den + A.c_num * (long long)len) * (long long)unc;
        if (lane == 0) {
            A.order[q0 + c] = j;
            A.uncached[q0 + j] = unc;
            A.ttft[q0 + j] = R - tj;
            if (A.completion) A.completion[q0 + j] = R;
            done[j >> 5] |= 1u << (j & 31);
        }
        __syncwarp();
        now = R; last = j; last_len = len; last_x = x;
    }
}

// ------------------------------------------------------------------------------------------------
// Trees with a budget: before and after the grouped loop.
// Before: the loop is all or nothing, so room for everything it can leave behind is checked first -- two nodes and one
// clock tick per prompt, and pool tokens for at most a budget's worth of new tokens plus three of alignment per node.
// After: the loop has kept the node arrays (parent, depth, length, children, stamps, dead flags) exact but has given
// the edges of new nodes virtual positions and has touched neither the token pool nor the child table.  Every node
// that is still alive gets its pool tokens (copied from the prompt that created its edge) and the child table is
// written afresh from the live nodes; nodes that were evicted again along the way cost nothing.
// ------------------------------------------------------------------------------------------------
struct LruInfo { long long n_nodes0; unsigned long long total_len; int32_t skip; int32_t pad; };

__global__ void lru_sum_kernel(const int64_t* __restrict__ off, int32_t n, LruInfo* info) {
    __shared__ unsigned long long s_w[8];
    const int32_t i = blockIdx.x * blockDim.x + threadIdx.x;
    unsigned long long x = i < n ? (unsigned long long)(off[i + 1] - off[i]) : 0ULL;
#pragma unroll
    for (int d = 16; d > 0; d >>= 1) x += __shfl_down_sync(FULL_MASK, x, d);
    if ((threadIdx.x & 31) == 0) s_w[threadIdx.x >> 5] = x;
    __syncthreads();
    if (threadIdx.x == 0) {
        unsigned long long t = 0;
        for (int w = 0; w < (int)(blockDim.x >> 5); ++w) t += s_w[w];
        atomicAdd(&info->total_len, t);
    }
}
__global__ void lru_check_kernel(TreeDev T, int32_t n, LruInfo* info) {
    TreeState* S = T.st;
    long long fresh = S->tokens_live + (long long)info->total_len;
    if (fresh > T.budget) fresh = T.budget;
    const bool ok = S->n_nodes + 2LL * n <= T.max_nodes && S->clock + (long long)n + 1 < T.max_clock &&
                    S->pool_used + fresh + 6LL * n + 16 <= T.max_pool;
    info->n_nodes0 = S->n_nodes;
    info->skip = ok ? 0 : 1;
    if (!ok) set_status(S, RT_ERR_CAPACITY, 115);
}

// One warp per node created by the loop: if it is alive and its edge has a virtual position, give it room in the pool
// and copy its tokens from the prompt that created the edge (decision c = the position's high bits; the edge holds
// that prompt's tokens from the node's depth on).
__global__ void __launch_bounds__(256)
lru_tokens_kernel(TreeDev T, const int32_t* __restrict__ order, const int32_t* __restrict__ qtok, const int64_t* __restrict__ qoff,
                  long long vbase, const LruInfo* info) {
    if (info->skip) return;
    const int lane = threadIdx.x & 31;
    const long long nwarps = ((long long)gridDim.x * blockDim.x) >> 5;
    const long long n_end = T.st->n_nodes;
    for (long long v = info->n_nodes0 + (((long long)blockIdx.x * blockDim.x + threadIdx.x) >> 5); v < n_end; v += nwarps) {
        if (T.dead[v]) continue;
        const long long so = T.span_off[v];
        if (so < vbase) continue;                           // a piece of an edge that was in the tree before: its tokens are in the pool
        const int32_t c = (int32_t)((so - vbase) >> 32), len = T.span_len[v], depth = T.depth_start[v];
        const int32_t* x = qtok + __ldg(qoff + __ldg(order + c)) + depth;
        long long base = 0;
        if (lane == 0) {
            const long long raw = (long long)atomicAdd((unsigned long long*)&T.st->pool_used, (unsigned long long)(len + 3));
            base = raw + (((long long)depth - raw) & 3LL);  // span_off = depth_start (mod 4), as everywhere
            if (raw + len + 3 > T.max_pool) { set_status(T.st, RT_ERR_CAPACITY, 116); base = -1; }      // (ruled out by the check before the loop)
        }
        base = __shfl_sync(FULL_MASK, base, 0);
        if (base < 0) continue;
        for (int32_t t = lane; t < len; t += 32) T.pool[base + t] = __ldg(x + t);
        if (lane == 0) T.span_off[v] = base;
    }
}

__global__ void table_clear_kernel(TreeDev T, const LruInfo* info) {
    if (info->skip) return;
    int4* p = reinterpret_cast<int4*>(T.table);
    const unsigned long long n16 = (T.table_mask + 1) * 2;              // an entry is two 16-byte units
    for (unsigned long long i = (unsigned long long)blockIdx.x * blockDim.x + threadIdx.x; i < n16; i += (unsigned long long)gridDim.x * blockDim.x)
        p[i] = make_int4(0, 0, 0, 0);
}

// One thread per node: every live node's first token, the mark at the end of its edge, and its entry in the (cleared)
// child table.
__global__ void lru_table_kernel(TreeDev T, long long vbase, const LruInfo* info) {
    if (info->skip) return;
    const long long v = (long long)blockIdx.x * blockDim.x + threadIdx.x;
    if (v < 1 || v >= T.st->n_nodes || T.dead[v]) return;
    const long long so = T.span_off[v];
    if (so >= vbase) return;                                // no room was found for it: the status word says so
    const int32_t len = T.span_len[v], ft = T.pool[so];
    T.first_tok[v] = ft;
    T.end_node[so + len - 1] = (int32_t)v;
    const unsigned long long key = make_key(T.parent[v], ft);
    unsigned long long slot = hash_key(key) & T.table_mask;
    for (unsigned long long pr = 0; pr <= T.table_mask; ++pr) {
        if (atomicCAS(&T.table[slot].key, 0ULL, key) == 0ULL) {
            T.table[slot].child = (int32_t)v; T.table[slot].span_len = len; T.table[slot].span_off = so; T.table[slot].chain_end = so + len;
            return;
        }
        slot = (slot + 1) & T.table_mask;
    }
    set_status(T.st, RT_ERR_CAPACITY, 117);
}

// batch size B: a query is finished when the last query of its bin of the processing order is
__global__ void batch_times_kernel(const int32_t* __restrict__ order, int32_t n, const int64_t* __restrict__ arrival,
                                   const int64_t* __restrict__ completion, int32_t n_queries, int32_t B, int64_t* ttft_b,
                                   int64_t* completion_b, int32_t* bad) {
    const int64_t i = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
    if (i >= n) return;
    int64_t last = (i / B + 1) * (int64_t)B - 1;
    if (last > n - 1) last = n - 1;
    const int32_t jl = __ldg(order + last), j = __ldg(order + i);
    if (jl < 0 || jl >= n_queries || j < 0 || j >= n_queries) {      // not a query: skipped, counted if the caller asked
        if (bad) atomicAdd(bad, 1);
        return;
    }
    const int64_t R = __ldg(completion + jl);
    completion_b[j] = R;
    ttft_b[j] = R - __ldg(arrival + j);
}

// klpm_replay through the grouped loop.  The order is checked first: the decisions that will be made are the entries
// before the first one that is not a query or names a query for the second time (the status word says so if there is
// one).  Slots are the queries in index order.
struct ReplayInfo { int32_t n_valid; int32_t pad; };
__global__ void replay_first_kernel(const int32_t* __restrict__ order, int32_t n_order, int32_t n_queries, int32_t* first_pos) {
    const int32_t p = blockIdx.x * blockDim.x + threadIdx.x;
    if (p >= n_order) return;
    const int32_t j = order[p];
    if (j >= 0 && j < n_queries) atomicMin(first_pos + j, p);
}
__global__ void replay_check_kernel(const int32_t* __restrict__ order, int32_t n_order, int32_t n_queries, const int64_t* __restrict__ off,
                                    const int32_t* __restrict__ first_pos, ReplayInfo* info, TreeState* st) {
    const int32_t p = blockIdx.x * blockDim.x + threadIdx.x;
    if (p >= n_order) return;
    const int32_t j = order[p];
    bool bad = j < 0 || j >= n_queries;
    if (!bad) { const int64_t len = off[j + 1] - off[j]; bad = len < 0 || len > 0x7fffffffLL || first_pos[j] < p; }
    if (bad) { atomicMin(&info->n_valid, p); set_status(st, RT_ERR_INVALID, 108); }
}
__global__ void replay_slots_kernel(const int64_t* __restrict__ arrival, int32_t n, long long* sorted_t, int32_t* ord) {
    const int32_t i = blockIdx.x * blockDim.x + threadIdx.x;
    if (i < n) { sorted_t[i] = arrival[i]; ord[i] = i; }
}
// the prompts a replay has processed, as the list the insertion after the loop works through (-1: not processed)
__global__ void replay_list_kernel(const int32_t* __restrict__ order, int32_t n_order, const ReplayInfo* info, int32_t* pend) {
    const int32_t p = blockIdx.x * blockDim.x + threadIdx.x;
    if (p < n_order) pend[p] = p < info->n_valid ? order[p] : -1;
}
__global__ void lru_sum_order_kernel(const int64_t* __restrict__ off, const int32_t* __restrict__ order, int32_t n_order,
                                     int32_t n_queries, LruInfo* info) {
    const int32_t p = blockIdx.x * blockDim.x + threadIdx.x;
    if (p >= n_order) return;
    const int32_t j = order[p];
    if (j >= 0 && j < n_queries) { const int64_t len = off[j + 1] - off[j]; if (len > 0) atomicAdd(&info->total_len, (unsigned long long)len); }
}

// slot order: bitonic sort of (arrival, index) pairs, padded to a power of two
__global__ void rank_init_kernel(const int64_t* __restrict__ arrival, int32_t n, long long np2, long long* key, int32_t* idx) {
    long long i = (long long)blockIdx.x * blockDim.x + threadIdx.x;
    if (i >= np2) return;
    key[i] = i < n ? arrival[i] : 0x7fffffffffffffffLL;
    idx[i] = i < n ? (int32_t)i : 0x7fffffff;
}
__global__ void slot_arrays_kernel(const int32_t* __restrict__ ord, const int64_t* __restrict__ off, int32_t n, long long* soff, int32_t* slen) {
    int32_t r = blockIdx.x * blockDim.x + threadIdx.x;
    if (r >= n) return;
    const int32_t qi = ord[r];
    const int64_t lo = off[qi];
    soff[r] = lo;
    slen[r] = (int32_t)(off[qi + 1] - lo);
}
__global__ void prio_init_kernel(const int64_t* __restrict__ prio, const int32_t* __restrict__ ord, int32_t n, long long np2,
                                 long long* key, int32_t* idx) {
    long long i = (long long)blockIdx.x * blockDim.x + threadIdx.x;
    if (i >= np2) return;
    key[i] = i < n ? prio[ord[i]] : 0x7fffffffffffffffLL;      // slot i holds query ord[i]
    idx[i] = i < n ? (int32_t)i : 0x7fffffff;
}
__global__ void prio_rank_kernel(const int32_t* __restrict__ pinv, int32_t n, int32_t* prank) {
    int32_t r = blockIdx.x * blockDim.x + threadIdx.x;
    if (r < n) prank[pinv[r]] = r;
}
__global__ void bitonic_step_kernel(long long* key, int32_t* idx, long long np2, long long k, long long j) {
    long long i = (long long)blockIdx.x * blockDim.x + threadIdx.x;
    if (i >= np2) return;
    long long l = i ^ j;
    if (l > i) {
        long long ki = key[i], kl = key[l];
        int32_t ii = idx[i], il = idx[l];
        bool gt = ki > kl || (ki == kl && ii > il);
        bool up = (i & k) == 0;
        if (gt == up) { key[i] = kl; key[l] = ki; idx[i] = il; idx[l] = ii; }
    }
}

// Two steps of one stage in one pass (partner distances j and j / 2): a thread holds the four entries that differ in
// those two bits.
__global__ void bitonic_step2_kernel(long long* key, int32_t* idx, long long np2, long long k, long long j) {
    const long long u = (long long)blockIdx.x * blockDim.x + threadIdx.x;
    if (u >= (np2 >> 2)) return;
    const long long j2 = j >> 1;
    const long long i0 = ((u & ~(j2 - 1)) << 2) | (u & (j2 - 1));      // u's bits with the two (adjacent) bit positions left out
    long long kk[4]; int32_t ii[4];
    const long long pos[4] = {i0, i0 | j2, i0 | j, i0 | j | j2};
#pragma unroll
    for (int r = 0; r < 4; ++r) { kk[r] = key[pos[r]]; ii[r] = idx[pos[r]]; }
    const bool up = (i0 & k) == 0;
    auto cx = [&](int x, int y) {
        const bool gt = kk[x] > kk[y] || (kk[x] == kk[y] && ii[x] > ii[y]);
        if (gt == up) { const long long tk = kk[x]; kk[x] = kk[y]; kk[y] = tk; const int32_t ti = ii[x]; ii[x] = ii[y]; ii[y] = ti; }
    };
    cx(0, 2); cx(1, 3);
    cx(0, 1); cx(2, 3);
#pragma unroll
    for (int r = 0; r < 4; ++r) { key[pos[r]] = kk[r]; idx[pos[r]] = ii[r]; }
}

// The steps of the same sort whose partner distance fits a tile of 4,096 pairs, done in shared memory: all stages
// k_lo .. k_hi when those are at most the tile (the start of the sort), otherwise the tail (distances below the
// tile) of the one stage k_lo = k_hi.
#define KLPM_SORT_TILE 4096
__global__ void __launch_bounds__(1024)
bitonic_tile_kernel(long long* key, int32_t* idx, long long np2, long long k_lo, long long k_hi) {
    __shared__ long long sk[KLPM_SORT_TILE];
    __shared__ int32_t si[KLPM_SORT_TILE];
    const int T = np2 < KLPM_SORT_TILE ? (int)np2 : KLPM_SORT_TILE;
    const long long base = (long long)blockIdx.x * T;
    for (int u = threadIdx.x; u < T; u += blockDim.x) { sk[u] = key[base + u]; si[u] = idx[base + u]; }
    __syncthreads();
    for (long long k = k_lo; k <= k_hi; k <<= 1) {
        const long long jmax = (k >> 1) < (long long)(T >> 1) ? (k >> 1) : (long long)(T >> 1);
        for (int j = (int)jmax; j > 0; j >>= 1) {
            for (int u = threadIdx.x; u < (T >> 1); u += blockDim.x) {
                const int i = ((u & ~(j - 1)) << 1) | (u & (j - 1)), l = i | j;      // the u-th pair at distance j
                const long long ki = sk[i], kl = sk[l];
                const int32_t ii = si[i], il = si[l];
                const bool gt = ki > kl || (ki == kl && ii > il);
                const bool up = ((base + i) & k) == 0;
                if (gt == up) { sk[i] = kl; sk[l] = ki; si[i] = il; si[l] = ii; }
            }
            __syncthreads();
        }
    }
    for (int u = threadIdx.x; u < T; u += blockDim.x) { key[base + u] = sk[u]; idx[base + u] = si[u]; }
}

// (key, idx) pairs ascending by key, then idx; np2 a power of two
void sort_pairs(long long* key, int32_t* idx, long long np2, cudaStream_t s) {
    const long long T = np2 < KLPM_SORT_TILE ? np2 : KLPM_SORT_TILE;
    const unsigned tiles = (unsigned)(np2 / T), blocks = (unsigned)((np2 + 255) / 256);
    const unsigned blocks4 = (unsigned)(((np2 >> 2) + 255) / 256);
    if (T >= 2) bitonic_tile_kernel<<<tiles, 1024, 0, s>>>(key, idx, np2, 2, T);
    for (long long k = T << 1; k <= np2; k <<= 1) {
        long long j = k >> 1;
        for (; (j >> 1) >= T; j >>= 2) bitonic_step2_kernel<<<blocks4, 256, 0, s>>>(key, idx, np2, k, j);
        if (j >= T) bitonic_step_kernel<<<blocks, 256, 0, s>>>(key, idx, np2, k, j);
        bitonic_tile_kernel<<<tiles, 1024, 0, s>>>(key, idx, np2, k, k);
    }
}

}  // namespace

// ====================================================================================================
// host side
// ====================================================================================================
struct rt_tree {
    rt_config cfg;
    TreeDev dev;
    int device;
    cudaStream_t last_stream;
    unsigned long long* match_counter;
    // batched match: the order in which queries are taken (bucketed by first token)
    long long match_cap;    // queries the three arrays below hold
    int32_t* match_perm; unsigned short* match_bucket; unsigned int* match_hist;
    // match records (MatchState): which match call wrote the caller's, and the library's own for klpm_run without one
    unsigned long long version;        // bumped by every call that changes the tree
    unsigned long long ms_tag, ms_version;
    const void *ms_state, *ms_tok, *ms_off;
    int32_t ms_n;
    MatchState* own_state; long long own_state_cap;
    // klpm_run scratch
    long long run_cap;      // slots allocated (power of two)
    long long* run_key; int32_t* run_ord; int32_t* run_m; int32_t* run_hint; long long* run_pos;
    long long* run_soff; int32_t* run_slen; int32_t* run_ntok;
    long long* run_pkey; int32_t* run_pinv; int32_t* run_prank;
    unsigned long long* run_partial; RunBcast* run_bc; RunSync* run_sy;
    // scratch of the grouped loop (trees without a budget)
    long long fast_cap;     // slots allocated (power of two)
    FDyn* fast_dyn; FStat* fast_stat; unsigned long long* fast_key_arr; int32_t* fast_mem;
    long long* fast_gh; int32_t* fast_gidx; unsigned int* fast_done; unsigned long long* fast_counter;
    long long* fast_lk; int32_t* fast_ls;
    FastPost* fast_post; long long* fast_bsum;
    long long fast_mem_cap;  // entries of fast_mem
    int32_t* lru_parked; LruInfo* lru_info;     // grouped loop on a tree with a budget
    int32_t* lru_hintc; long long lru_hintc_cap;
    int2* lru_leaf_run;
    ReplayInfo* replay_info;
    int run_path;           // which loop the last klpm_run took: 0 none yet, 1 one by one, 2 grouped
    int num_sms;
    int32_t* claim;         // bulk insertion: per-node claim words (0x7fffffff when idle)
    long long bulk_cap;     // bulk insertion: prompts its per-prompt scratch holds
    int32_t *bulk_pend_a, *bulk_pend_b, *bulk_pm, *bulk_pnode, *bulk_poff;
    BulkSync* bulk_sync;
    // checkpoint (rt_checkpoint / rt_rollback): copies of everything a later call can modify
    bool ck_valid;
    int32_t *ck_parent, *ck_depth_start, *ck_span_len, *ck_nchild, *ck_clock_owner, *ck_first_tok;
    int64_t *ck_span_off, *ck_last_access;
    uint8_t* ck_dead;
    Entry* ck_table;
    TreeState* ck_st;
};

namespace {

#define CK(call) do { cudaError_t e_ = (call); if (e_ != cudaSuccess) { \
    fprintf(stderr, "klpm: %s failed at %s:%d: %s\n", #call, __FILE__, __LINE__, cudaGetErrorString(e_)); return RT_ERR_CUDA; } } while (0)

template <typename P> rt_status dalloc(P** p, size_t count) {
    void* v = nullptr;
    CK(cudaMalloc(&v, count * sizeof(P) + 256));
    *p = (P*)v;
    return RT_OK;
}

void free_tree(rt_tree* t) {
    TreeDev& d = t->dev;
    cudaFree(d.parent); cudaFree(d.depth_start); cudaFree(d.span_len); cudaFree(d.nchild); cudaFree(d.first_tok);
    cudaFree(t->ck_first_tok);
    cudaFree(d.span_off); cudaFree(d.last_access); cudaFree(d.dead); cudaFree(d.clock_owner);
    cudaFree(d.table); cudaFree(d.pool); cudaFree(d.end_node); cudaFree(d.st); cudaFree(t->match_counter);
    cudaFree(t->match_perm); cudaFree(t->match_bucket); cudaFree(t->match_hist); cudaFree(t->own_state);
    cudaFree(t->run_key); cudaFree(t->run_ord); cudaFree(t->run_m); cudaFree(t->run_hint);
    cudaFree(t->run_pos); cudaFree(t->run_soff); cudaFree(t->run_slen); cudaFree(t->run_ntok);
    cudaFree(t->run_pkey); cudaFree(t->run_pinv); cudaFree(t->run_prank);
    cudaFree(t->run_partial); cudaFree(t->run_bc); cudaFree(t->run_sy);
    cudaFree(t->fast_dyn); cudaFree(t->fast_stat); cudaFree(t->fast_key_arr); cudaFree(t->fast_mem);
    cudaFree(t->fast_gh); cudaFree(t->fast_gidx); cudaFree(t->fast_done); cudaFree(t->fast_counter);
    cudaFree(t->fast_lk); cudaFree(t->fast_ls); cudaFree(t->fast_post); cudaFree(t->fast_bsum);
    cudaFree(t->lru_parked); cudaFree(t->lru_info); cudaFree(t->lru_hintc); cudaFree(t->lru_leaf_run); cudaFree(t->replay_info);
    cudaFree(t->claim);
    cudaFree(t->bulk_pend_a); cudaFree(t->bulk_pend_b); cudaFree(t->bulk_pm); cudaFree(t->bulk_pnode); cudaFree(t->bulk_poff);
    cudaFree(t->bulk_sync);
    cudaFree(t->ck_parent); cudaFree(t->ck_depth_start); cudaFree(t->ck_span_len); cudaFree(t->ck_nchild);
    cudaFree(t->ck_clock_owner); cudaFree(t->ck_span_off); cudaFree(t->ck_last_access); cudaFree(t->ck_dead);
    cudaFree(t->ck_table); cudaFree(t->ck_st);
    delete t;
}

rt_status ensure_run_scratch(rt_tree* t, long long n) {
    long long np2 = 1;
    while (np2 < n) np2 <<= 1;
    if (np2 <= t->run_cap) return RT_OK;
    cudaFree(t->run_key); cudaFree(t->run_ord); cudaFree(t->run_m); cudaFree(t->run_hint);
    cudaFree(t->run_pos); cudaFree(t->run_soff); cudaFree(t->run_slen); cudaFree(t->run_ntok);
    cudaFree(t->run_pkey); cudaFree(t->run_pinv); cudaFree(t->run_prank);
    t->run_ntok = nullptr; t->run_pkey = nullptr; t->run_pinv = nullptr; t->run_prank = nullptr;
    t->run_key = nullptr; t->run_ord = nullptr; t->run_m = nullptr; t->run_hint = nullptr; t->run_pos = nullptr;
    t->run_soff = nullptr; t->run_slen = nullptr;
    t->run_cap = 0;
    rt_status s;
    if ((s = dalloc(&t->run_key, np2))) return s;
    if ((s = dalloc(&t->run_ord, np2))) return s;
    if ((s = dalloc(&t->run_m, np2))) return s;
    if ((s = dalloc(&t->run_hint, np2))) return s;
    if ((s = dalloc(&t->run_pos, np2))) return s;
    if ((s = dalloc(&t->run_soff, np2))) return s;
    if ((s = dalloc(&t->run_slen, np2))) return s;
    if ((s = dalloc(&t->run_ntok, np2))) return s;
    if ((s = dalloc(&t->run_pkey, np2))) return s;
    if ((s = dalloc(&t->run_pinv, np2))) return s;
    if ((s = dalloc(&t->run_prank, np2))) return s;
    t->run_cap = np2;
    return RT_OK;
}

rt_status ensure_fast_scratch(rt_tree* t, long long n) {
    long long np2 = 1;
    while (np2 < n) np2 <<= 1;
    if (np2 <= t->fast_cap) return RT_OK;
    cudaFree(t->fast_dyn); cudaFree(t->fast_stat); cudaFree(t->fast_key_arr); cudaFree(t->fast_mem);
    cudaFree(t->fast_gh); cudaFree(t->fast_gidx); cudaFree(t->fast_done); cudaFree(t->fast_counter);
    cudaFree(t->fast_lk); cudaFree(t->fast_ls);
    t->fast_lk = nullptr; t->fast_ls = nullptr;
    t->fast_dyn = nullptr; t->fast_stat = nullptr; t->fast_key_arr = nullptr; t->fast_mem = nullptr;
    t->fast_gh = nullptr; t->fast_gidx = nullptr; t->fast_done = nullptr; t->fast_counter = nullptr;
    t->fast_cap = 0;
    rt_status s;
    if ((s = dalloc(&t->fast_dyn, np2))) return s;
    if ((s = dalloc(&t->fast_stat, np2))) return s;
    if ((s = dalloc(&t->fast_key_arr, np2))) return s;
    // trees with a budget: groups formed by evictions are appended behind the first n entries
    t->fast_mem_cap = t->cfg.budget_tokens > 0 ? np2 + (8 * np2 > (1LL << 20) ? 8 * np2 : (1LL << 20)) : np2;
    if ((s = dalloc(&t->fast_mem, t->fast_mem_cap))) return s;
    if ((s = dalloc(&t->fast_gh, np2))) return s;
    if ((s = dalloc(&t->fast_gidx, np2))) return s;
    if ((s = dalloc(&t->fast_done, 3 * (np2 / 32 + 32)))) return s;     // processed bitmap, grouped bitmap, passed-over bitmap
    if ((s = dalloc(&t->fast_lk, np2))) return s;
    if ((s = dalloc(&t->fast_ls, np2))) return s;
    if (!t->fast_post && (s = dalloc(&t->fast_post, 1))) return s;
    if (!t->fast_bsum && (s = dalloc(&t->fast_bsum, 1024))) return s;
    t->fast_cap = np2;
    return RT_OK;
}

bool params_ok(const klpm_params* p) {
    return p && p->policy >= KLPM_POLICY_FCFS && p->policy <= KLPM_POLICY_KLPM && p->k >= 1 && p->c_den >= 1 && p->c_num >= 0;
}

// Settings for tests and debugging (klpm_debug_set); process-wide, read when a call is made.
struct DebugKnobs {
    long long run_one_by_one;     // 1: trees without a budget take the one-by-one loop too
    long long fast_max_blocks;    // grouped loop: most tournament leaf blocks (0 = the built-in 8,192)
    long long fast_smem_kb;       // grouped loop: shared memory it may use (0 = the built-in 224 KB)
    long long wait_limit_ns;      // one-by-one loop: limit of a hand-over wait
};
DebugKnobs g_knobs = {0, 0, 0, KLPM_WAIT_LIMIT_NS};

SelectScratch* g_select_scratch[64] = {nullptr};
TopkScratch* g_topk_scratch[64] = {nullptr};
StaticSelectScratch* g_select_static_addr[64] = {nullptr};   // device address of g_select_static, per device

// Many prompts at once into a tree without a budget (see the bulk kernels).  Waits for the stream once per round.
rt_status ensure_bulk_scratch(rt_tree* t, int32_t n) {
    rt_status st = RT_OK;
    if (n > t->bulk_cap) {                     // per-prompt scratch, kept for later calls
        cudaFree(t->bulk_pend_a); cudaFree(t->bulk_pend_b); cudaFree(t->bulk_pm); cudaFree(t->bulk_pnode); cudaFree(t->bulk_poff);
        t->bulk_pend_a = t->bulk_pend_b = t->bulk_pm = t->bulk_pnode = t->bulk_poff = nullptr;
        t->bulk_cap = 0;
        if ((st = dalloc(&t->bulk_pend_a, n)) || (st = dalloc(&t->bulk_pend_b, n)) || (st = dalloc(&t->bulk_pm, n)) ||
            (st = dalloc(&t->bulk_pnode, n)) || (st = dalloc(&t->bulk_poff, n))) return st;
        t->bulk_cap = n;
    }
    if (!t->bulk_sync && (st = dalloc(&t->bulk_sync, 1))) return st;        // list lengths, work counter, grid barrier
    return RT_OK;
}

// `state` (nullable): records of a batched match of these prompts against the tree as it is now; the first round
// then needs no walk.  Everything is enqueued on `s`; nothing waits for the device.
// `list_ready`: bulk_pend_a already holds the n prompts to store (entries < 0 are skipped) and *n_total_dev how many they are.
rt_status bulk_insert(rt_tree* t, const int32_t* d_tokens, const int64_t* d_offsets, int32_t n, cudaStream_t s,
                      const MatchState* state = nullptr, unsigned long long tag = 0, bool list_ready = false,
                      const int32_t* n_total_dev = nullptr) {
    rt_status st = ensure_bulk_scratch(t, n);
    if (st) return st;
    BulkSync* g = t->bulk_sync;
    // claim words start idle (an earlier call that ran out of capacity may have left some set)
    bulk_fill_kernel<<<(unsigned)((t->dev.max_nodes + 255) / 256), 256, 0, s>>>(t->claim, t->dev.max_nodes, 0x7fffffff);
    if (!list_ready) bulk_iota_kernel<<<(unsigned)((n + 255) / 256), 256, 0, s>>>(t->bulk_pend_a, n);
    CK(cudaMemsetAsync(g, 0, sizeof(BulkSync), s));
    BulkArgs a;
    a.tok = d_tokens; a.off = d_offsets; a.pend_in = t->bulk_pend_a; a.pend_out = t->bulk_pend_b; a.n_out = &g->cnt_w[0];
    a.pend_next = t->bulk_pend_a; a.n_next = &g->cnt_a[0]; a.n_walk = &g->n_walk;      // the walk has consumed pend_a by the time apply refills it
    a.claim = t->claim; a.pm = t->bulk_pm; a.pnode = t->bulk_pnode; a.poff = t->bulk_poff;
    long long blocks = ((long long)n + 7) / 8;
    if (blocks > (long long)t->num_sms * 8) blocks = (long long)t->num_sms * 8;
    // the first round: every prompt from the root (or from its match record), then cuts and leaves
    if (state) bulk_from_state_kernel<<<(unsigned)blocks, 256, 0, s>>>(t->dev, a, state, tag, (unsigned)n);
    else bulk_walk_kernel<<<(unsigned)blocks, 256, 0, s>>>(t->dev, a, (unsigned)n);
    bulk_apply_kernel<<<(unsigned)blocks, 256, 0, s>>>(t->dev, a);
    CK(cudaGetLastError());
    // every later round, and the clock, in one cooperative kernel
    int per_sm = 0;
    CK(cudaOccupancyMaxActiveBlocksPerMultiprocessor(&per_sm, bulk_rounds_kernel, 256, 0));
    if (per_sm < 1) return RT_ERR_CUDA;
    const unsigned grid = (unsigned)t->num_sms * (unsigned)(per_sm < 2 ? per_sm : 2);
    long long n_total = n, limit = g_knobs.wait_limit_ns;
    void* kargs[] = {(void*)&t->dev, (void*)&a, (void*)&g, (void*)&n_total, (void*)&n_total_dev, (void*)&limit};
    CK(cudaLaunchCooperativeKernel((void*)bulk_rounds_kernel, dim3(grid), dim3(256), kargs, 0, s));
    return RT_OK;
}

#define KLPM_ORDER_MIN 2048       // smaller batches are matched in index order (three launches saved)
std::atomic<unsigned long long> g_match_tag{0};

// The batched match: the order in which the queries are taken, then the kernel.  `state` (nullable) receives the
// per-query records, stamped with `tag`.
rt_status launch_match(rt_tree* t, const int32_t* d_q_tokens, const int64_t* d_q_offsets, int32_t nq, int32_t* d_match_len,
                       int32_t* d_term_node, int32_t* d_term_off, MatchState* state, unsigned long long tag, cudaStream_t s) {
    const int32_t* perm = nullptr;
    if (nq >= KLPM_ORDER_MIN) {
        if (nq > t->match_cap) {
            cudaFree(t->match_perm); cudaFree(t->match_bucket);
            t->match_perm = nullptr; t->match_bucket = nullptr; t->match_cap = 0;
            rt_status st;
            if ((st = dalloc(&t->match_perm, nq)) || (st = dalloc(&t->match_bucket, nq))) return st;
            t->match_cap = nq;
        }
        if (!t->match_hist) { rt_status st = dalloc(&t->match_hist, KLPM_ORDER_BUCKETS); if (st) return st; }
        const unsigned qb = (unsigned)((nq + 255) / 256);
        CK(cudaMemsetAsync(t->match_hist, 0, KLPM_ORDER_BUCKETS * sizeof(unsigned int), s));
        order_hist_kernel<<<qb, 256, 0, s>>>(d_q_tokens, d_q_offsets, nq, t->match_hist, t->match_bucket);
        order_scan_kernel<<<1, 1024, 0, s>>>(t->match_hist);
        order_scatter_kernel<<<qb, 256, 0, s>>>(t->match_bucket, nq, t->match_hist, t->match_perm);
        perm = t->match_perm;
    }
    CK(cudaMemsetAsync(t->match_counter, 0, sizeof(unsigned long long), s));
    const int threads = 256, warps_per_block = threads / 32;
    long long blocks = ((long long)nq + warps_per_block - 1) / warps_per_block;
    const long long max_blocks = (long long)t->num_sms * 8;
    if (blocks > max_blocks) blocks = max_blocks;
    if (t->cfg.budget_tokens == 0) {
        if (state) match_chain_kernel<true><<<(unsigned)blocks, threads, 0, s>>>(t->dev, d_q_tokens, d_q_offsets, nq, perm, d_match_len,
                                                                               d_term_node, d_term_off, state, tag, t->match_counter);
        else match_chain_kernel<false><<<(unsigned)blocks, threads, 0, s>>>(t->dev, d_q_tokens, d_q_offsets, nq, perm, d_match_len,
                                                                            d_term_node, d_term_off, nullptr, 0ULL, t->match_counter);
    } else {
        match_batch_kernel<<<(unsigned)blocks, threads, 0, s>>>(t->dev, d_q_tokens, d_q_offsets, nq, perm, d_match_len,
                                                               d_term_node, d_term_off, state, tag, t->match_counter);
    }
    CK(cudaGetLastError());
    return RT_OK;
}

}  // namespace

extern "C" {

int32_t klpm_abi_version(void) { return KLPM_ABI_VERSION; }

rt_status rt_create(const rt_config* cfg, rt_tree** out) {
    if (!cfg || !out || cfg->max_nodes < 2 || cfg->max_pool_tokens < 1 || cfg->budget_tokens < 0 ||
        cfg->max_nodes > 0x7ffffff0LL || cfg->max_clock < 0) return RT_ERR_INVALID;
    rt_tree* t = new (std::nothrow) rt_tree();
    if (!t) return RT_ERR_CUDA;
    memset(t, 0, sizeof(*t));
    t->cfg = *cfg;
    CK(cudaGetDevice(&t->device));
    CK(cudaDeviceGetAttribute(&t->num_sms, cudaDevAttrMultiProcessorCount, t->device));
    TreeDev& d = t->dev;
    d.max_nodes = cfg->max_nodes;
    d.max_pool = cfg->max_pool_tokens;
    d.max_clock = (cfg->max_clock > 0 ? cfg->max_clock : cfg->max_nodes) + 2;
    d.budget = cfg->budget_tokens;
    unsigned long long cap = 1024;
    while (cap < 2ULL * (unsigned long long)cfg->max_nodes) cap <<= 1;
    d.table_mask = cap - 1;
    rt_status s = RT_OK;
    if ((s = dalloc(&d.parent, d.max_nodes)) || (s = dalloc(&d.depth_start, d.max_nodes)) ||
        (s = dalloc(&d.span_len, d.max_nodes)) || (s = dalloc(&d.nchild, d.max_nodes)) || (s = dalloc(&d.first_tok, d.max_nodes)) ||
        (s = dalloc(&d.span_off, d.max_nodes)) || (s = dalloc(&d.last_access, d.max_nodes)) ||
        (s = dalloc(&d.dead, d.max_nodes)) || (s = dalloc(&d.clock_owner, d.max_clock)) ||
        (s = dalloc(&d.table, cap)) || (s = dalloc(&d.pool, d.max_pool)) || (s = dalloc(&d.st, 1)) ||
        (s = dalloc(&d.end_node, d.max_pool)) ||
        (s = dalloc(&t->match_counter, 1)) || (s = dalloc(&t->run_partial, 1024)) || (s = dalloc(&t->run_bc, 1)) || (s = dalloc(&t->run_sy, 1)) ||
        (s = dalloc(&t->claim, d.max_nodes))) {
        free_tree(t);
        return s;
    }
    // root: node 0, empty edge
    cudaError_t e = cudaMemset(d.table, 0, cap * sizeof(Entry));
    if (e == cudaSuccess) e = cudaMemset(d.end_node, 0xff, d.max_pool * sizeof(int32_t) + 256);
    if (e == cudaSuccess) e = cudaMemset(d.clock_owner, 0, d.max_clock * sizeof(int32_t));
    if (e == cudaSuccess) e = cudaMemset(d.parent, 0, sizeof(int32_t));
    if (e == cudaSuccess) e = cudaMemset(d.depth_start, 0, sizeof(int32_t));
    if (e == cudaSuccess) e = cudaMemset(d.span_len, 0, sizeof(int32_t));
    if (e == cudaSuccess) e = cudaMemset(d.nchild, 0, sizeof(int32_t));
    if (e == cudaSuccess) e = cudaMemset(d.first_tok, 0, sizeof(int32_t));
    if (e == cudaSuccess) e = cudaMemset(d.span_off, 0, sizeof(int64_t));
    if (e == cudaSuccess) e = cudaMemset(d.last_access, 0, sizeof(int64_t));
    if (e == cudaSuccess) e = cudaMemset(d.dead, 0, 1);
    if (e == cudaSuccess) {
        bulk_fill_kernel<<<(unsigned)((d.max_nodes + 255) / 256), 256>>>(t->claim, d.max_nodes, 0x7fffffff);
        e = cudaGetLastError();
    }
    TreeState st0;
    memset(&st0, 0, sizeof(st0));
    st0.n_nodes = 1;
    st0.lru_cursor = 1;
    if (e == cudaSuccess) e = cudaMemcpy(d.st, &st0, sizeof(st0), cudaMemcpyHostToDevice);
    if (e == cudaSuccess) e = cudaDeviceSynchronize();
    if (e != cudaSuccess) {
        fprintf(stderr, "klpm: tree initialisation failed: %s\n", cudaGetErrorString(e));
        free_tree(t);
        return RT_ERR_CUDA;
    }
    *out = t;
    return RT_OK;
}

rt_status rt_destroy(rt_tree* tree) {
    if (!tree) return RT_ERR_INVALID;
    cudaDeviceSynchronize();
    free_tree(tree);
    return RT_OK;
}

rt_status rt_insert(rt_tree* tree, const int32_t* d_tokens, const int64_t* d_offsets, int32_t n,
                    int32_t* d_new_tokens, void* stream) {
    if (!tree || n < 0 || (n > 0 && (!d_tokens || !d_offsets))) return RT_ERR_INVALID;
    if (n == 0) return RT_OK;
    tree->version++;
    if (!d_new_tokens && tree->cfg.budget_tokens == 0 && n >= 64) {
        tree->last_stream = (cudaStream_t)stream;
        return bulk_insert(tree, d_tokens, d_offsets, n, (cudaStream_t)stream);
    }
    SeqArgs a;
    memset(&a, 0, sizeof(a));
    a.tok = d_tokens; a.off = d_offsets; a.n = n; a.n_queries = n; a.new_tokens = d_new_tokens; a.c_den = 1;
    tree->last_stream = (cudaStream_t)stream;
    sequential_kernel<<<1, 1024, 0, (cudaStream_t)stream>>>(tree->dev, a);
    CK(cudaGetLastError());
    return RT_OK;
}

rt_status rt_build(const int32_t* d_tokens, const int64_t* d_offsets, int32_t n_prompts, const rt_config* cfg,
                   void* stream, rt_tree** out) {
    if (!out || n_prompts < 0) return RT_ERR_INVALID;
    rt_tree* t = nullptr;
    rt_status s = rt_create(cfg, &t);
    if (s) return s;
    s = rt_insert(t, d_tokens, d_offsets, n_prompts, nullptr, stream);
    if (s) { rt_destroy(t); return s; }
    *out = t;
    return RT_OK;
}

rt_status rt_match_batch_ex(rt_tree* tree, const int32_t* d_q_tokens, const int64_t* d_q_offsets, int32_t nq,
                            int32_t* d_match_len, int32_t* d_term_node, int32_t* d_term_off, klpm_match_state* d_state,
                            void* stream) {
    if (!tree || nq < 0 || (nq > 0 && (!d_q_tokens || !d_q_offsets || !d_match_len))) return RT_ERR_INVALID;
    if (nq == 0) return RT_OK;
    cudaStream_t s = (cudaStream_t)stream;
    tree->last_stream = s;
    unsigned long long tag = 0;
    if (d_state) {
        tag = ++g_match_tag;
        tree->ms_tag = tag; tree->ms_version = tree->version; tree->ms_state = d_state; tree->ms_tok = d_q_tokens;
        tree->ms_off = d_q_offsets; tree->ms_n = nq;
    }
    return launch_match(tree, d_q_tokens, d_q_offsets, nq, d_match_len, d_term_node, d_term_off,
                        reinterpret_cast<MatchState*>(d_state), tag, s);
}

rt_status rt_match_batch(const rt_tree* tree, const int32_t* d_q_tokens, const int64_t* d_q_offsets, int32_t nq,
                         int32_t* d_match_len, int32_t* d_term_node, int32_t* d_term_off, void* stream) {
    return rt_match_batch_ex(const_cast<rt_tree*>(tree), d_q_tokens, d_q_offsets, nq, d_match_len, d_term_node, d_term_off,
                             nullptr, stream);
}

rt_status rt_stats(rt_tree* tree, int64_t* n_nodes, int64_t* n_tokens, int64_t* clock, int64_t* evictions, int64_t* pool_used) {
    if (!tree) return RT_ERR_INVALID;
    CK(cudaStreamSynchronize(tree->last_stream));
    TreeState st;
    CK(cudaMemcpy(&st, tree->dev.st, sizeof(st), cudaMemcpyDeviceToHost));
    if (n_nodes) *n_nodes = st.live_nodes;
    if (n_tokens) *n_tokens = st.tokens_live;
    if (clock) *clock = st.clock;
    if (evictions) *evictions = st.evictions;
    if (pool_used) *pool_used = st.pool_used;
    return RT_OK;
}

rt_status rt_clone(rt_tree* tree, void* stream, rt_tree** out) {
    if (!tree || !out) return RT_ERR_INVALID;
    rt_tree* c = nullptr;
    rt_status s = rt_create(&tree->cfg, &c);
    if (s) return s;
    const TreeDev& a = tree->dev;
    TreeDev& b = c->dev;
    const unsigned long long cap = a.table_mask + 1;
    cudaStream_t st = (cudaStream_t)stream;
    tree->last_stream = st;
    c->last_stream = st;
    const cudaMemcpyKind k = cudaMemcpyDeviceToDevice;
    cudaError_t e = cudaMemcpyAsync(b.parent, a.parent, a.max_nodes * sizeof(int32_t), k, st);
    if (e == cudaSuccess) e = cudaMemcpyAsync(b.depth_start, a.depth_start, a.max_nodes * sizeof(int32_t), k, st);
    if (e == cudaSuccess) e = cudaMemcpyAsync(b.span_len, a.span_len, a.max_nodes * sizeof(int32_t), k, st);
    if (e == cudaSuccess) e = cudaMemcpyAsync(b.nchild, a.nchild, a.max_nodes * sizeof(int32_t), k, st);
    if (e == cudaSuccess) e = cudaMemcpyAsync(b.first_tok, a.first_tok, a.max_nodes * sizeof(int32_t), k, st);
    if (e == cudaSuccess) e = cudaMemcpyAsync(b.span_off, a.span_off, a.max_nodes * sizeof(int64_t), k, st);
    if (e == cudaSuccess) e = cudaMemcpyAsync(b.last_access, a.last_access, a.max_nodes * sizeof(int64_t), k, st);
    if (e == cudaSuccess) e = cudaMemcpyAsync(b.dead, a.dead, a.max_nodes, k, st);
    if (e == cudaSuccess) e = cudaMemcpyAsync(b.clock_owner, a.clock_owner, a.max_clock * sizeof(int32_t), k, st);
    if (e == cudaSuccess) e = cudaMemcpyAsync(b.table, a.table, cap * sizeof(Entry), k, st);
    if (e == cudaSuccess) e = cudaMemcpyAsync(b.pool, a.pool, a.max_pool * sizeof(int32_t), k, st);
    if (e == cudaSuccess) e = cudaMemcpyAsync(b.end_node, a.end_node, a.max_pool * sizeof(int32_t), k, st);
    if (e == cudaSuccess) e = cudaMemcpyAsync(b.st, a.st, sizeof(TreeState), k, st);
    if (e != cudaSuccess) {
        fprintf(stderr, "klpm: rt_clone failed: %s\n", cudaGetErrorString(e));
        cudaStreamSynchronize(st);
        free_tree(c);
        return RT_ERR_CUDA;
    }
    *out = c;
    return RT_OK;
}

rt_status rt_checkpoint(rt_tree* tree, void* stream) {
    if (!tree) return RT_ERR_INVALID;
    TreeDev& d = tree->dev;
    const unsigned long long cap = d.table_mask + 1;
    rt_status s = RT_OK;
    if (!tree->ck_parent) {
        if ((s = dalloc(&tree->ck_parent, d.max_nodes)) || (s = dalloc(&tree->ck_depth_start, d.max_nodes)) ||
            (s = dalloc(&tree->ck_span_len, d.max_nodes)) || (s = dalloc(&tree->ck_nchild, d.max_nodes)) ||
            (s = dalloc(&tree->ck_first_tok, d.max_nodes)) ||
            (s = dalloc(&tree->ck_span_off, d.max_nodes)) || (s = dalloc(&tree->ck_last_access, d.max_nodes)) ||
            (s = dalloc(&tree->ck_dead, d.max_nodes)) || (s = dalloc(&tree->ck_clock_owner, d.max_clock)) ||
            (s = dalloc(&tree->ck_table, cap)) || (s = dalloc(&tree->ck_st, 1))) return s;
    }
    cudaStream_t st = (cudaStream_t)stream;
    tree->last_stream = st;
    const cudaMemcpyKind k = cudaMemcpyDeviceToDevice;
    CK(cudaMemcpyAsync(tree->ck_parent, d.parent, d.max_nodes * sizeof(int32_t), k, st));
    CK(cudaMemcpyAsync(tree->ck_depth_start, d.depth_start, d.max_nodes * sizeof(int32_t), k, st));
    CK(cudaMemcpyAsync(tree->ck_span_len, d.span_len, d.max_nodes * sizeof(int32_t), k, st));
    CK(cudaMemcpyAsync(tree->ck_nchild, d.nchild, d.max_nodes * sizeof(int32_t), k, st));
    CK(cudaMemcpyAsync(tree->ck_first_tok, d.first_tok, d.max_nodes * sizeof(int32_t), k, st));
    CK(cudaMemcpyAsync(tree->ck_span_off, d.span_off, d.max_nodes * sizeof(int64_t), k, st));
    CK(cudaMemcpyAsync(tree->ck_last_access, d.last_access, d.max_nodes * sizeof(int64_t), k, st));
    CK(cudaMemcpyAsync(tree->ck_dead, d.dead, d.max_nodes, k, st));
    CK(cudaMemcpyAsync(tree->ck_clock_owner, d.clock_owner, d.max_clock * sizeof(int32_t), k, st));
    CK(cudaMemcpyAsync(tree->ck_table, d.table, cap * sizeof(Entry), k, st));
    CK(cudaMemcpyAsync(tree->ck_st, d.st, sizeof(TreeState), k, st));
    tree->ck_valid = true;
    return RT_OK;
}

rt_status rt_rollback(rt_tree* tree, void* stream) {
    if (!tree || !tree->ck_valid) return RT_ERR_INVALID;
    tree->version++;
    TreeDev& d = tree->dev;
    const unsigned long long cap = d.table_mask + 1;
    cudaStream_t st = (cudaStream_t)stream;
    tree->last_stream = st;
    const cudaMemcpyKind k = cudaMemcpyDeviceToDevice;
    CK(cudaMemcpyAsync(d.parent, tree->ck_parent, d.max_nodes * sizeof(int32_t), k, st));
    CK(cudaMemcpyAsync(d.depth_start, tree->ck_depth_start, d.max_nodes * sizeof(int32_t), k, st));
    CK(cudaMemcpyAsync(d.span_len, tree->ck_span_len, d.max_nodes * sizeof(int32_t), k, st));
    CK(cudaMemcpyAsync(d.nchild, tree->ck_nchild, d.max_nodes * sizeof(int32_t), k, st));
    CK(cudaMemcpyAsync(d.first_tok, tree->ck_first_tok, d.max_nodes * sizeof(int32_t), k, st));
    CK(cudaMemcpyAsync(d.span_off, tree->ck_span_off, d.max_nodes * sizeof(int64_t), k, st));
    CK(cudaMemcpyAsync(d.last_access, tree->ck_last_access, d.max_nodes * sizeof(int64_t), k, st));
    CK(cudaMemcpyAsync(d.dead, tree->ck_dead, d.max_nodes, k, st));
    CK(cudaMemcpyAsync(d.clock_owner, tree->ck_clock_owner, d.max_clock * sizeof(int32_t), k, st));
    CK(cudaMemcpyAsync(d.table, tree->ck_table, cap * sizeof(Entry), k, st));
    CK(cudaMemcpyAsync(d.st, tree->ck_st, sizeof(TreeState), k, st));
    return RT_OK;
}

rt_status rt_status_detail(rt_tree* tree, int32_t* detail) {
    if (!tree || !detail) return RT_ERR_INVALID;
    CK(cudaStreamSynchronize(tree->last_stream));
    TreeState st;
    CK(cudaMemcpy(&st, tree->dev.st, sizeof(st), cudaMemcpyDeviceToHost));
    *detail = st.detail;
    return RT_OK;
}

rt_status rt_sync_status(rt_tree* tree, void* stream) {
    if (!tree) return RT_ERR_INVALID;
    CK(cudaStreamSynchronize((cudaStream_t)stream));
    TreeState st;
    CK(cudaMemcpy(&st, tree->dev.st, sizeof(st), cudaMemcpyDeviceToHost));
    return (rt_status)st.status;
}

rt_status klpm_select(const int32_t* d_match_len, const int64_t* d_arrival, const uint8_t* d_waiting, int32_t nq,
                      int64_t pick_counter, const klpm_params* params, int32_t* d_pick, void* stream) {
    if (!params_ok(params) || nq < 0 || !d_pick || pick_counter < 0 ||
        (nq > 0 && (!d_match_len || !d_arrival || !d_waiting))) return RT_ERR_INVALID;
    int dev = 0;
    CK(cudaGetDevice(&dev));
    if (dev < 0 || dev >= 64) return RT_ERR_INVALID;
    if (!g_select_scratch[dev]) {
        SelectScratch* p = nullptr;
        CK(cudaMalloc((void**)&p, sizeof(SelectScratch)));
        CK(cudaMemset(p, 0, sizeof(SelectScratch)));
        g_select_scratch[dev] = p;
    }
    const bool fcfs_turn = params->policy == KLPM_POLICY_FCFS ||
                           (params->policy == KLPM_POLICY_KLPM && pick_counter % params->k == 0);
    long long blocks = ((long long)nq + 2047) / 2048;
    if (blocks < 1) blocks = 1;
    if (blocks > 1024) blocks = 1024;
    cudaStream_t s = (cudaStream_t)stream;
    if (fcfs_turn) select_kernel<false><<<(unsigned)blocks, 512, 0, s>>>(d_match_len, d_arrival, d_waiting, nq, d_pick, g_select_scratch[dev]);
    else select_kernel<true><<<(unsigned)blocks, 512, 0, s>>>(d_match_len, d_arrival, d_waiting, nq, d_pick, g_select_scratch[dev]);
    CK(cudaGetLastError());
    return RT_OK;
}

rt_status klpm_select_topk(const int32_t* d_match_len, const int64_t* d_arrival, const uint8_t* d_waiting, int32_t nq,
                           int32_t kk, int32_t* d_out, void* stream) {
    if (nq < 0 || kk < 1 || kk > KLPM_TOPK_MAX || !d_out || (nq > 0 && (!d_match_len || !d_arrival || !d_waiting))) return RT_ERR_INVALID;
    int dev = 0;
    CK(cudaGetDevice(&dev));
    if (dev < 0 || dev >= 64) return RT_ERR_INVALID;
    if (!g_topk_scratch[dev]) {
        TopkScratch* p = nullptr;
        CK(cudaMalloc((void**)&p, sizeof(TopkScratch)));
        CK(cudaMemset(p, 0, sizeof(TopkScratch)));
        g_topk_scratch[dev] = p;
    }
    long long blocks = ((long long)nq + 4095) / 4096;
    if (blocks < 1) blocks = 1;
    if (blocks > KLPM_TOPK_BLOCKS) blocks = KLPM_TOPK_BLOCKS;
    select_topk_kernel<<<(unsigned)blocks, 512, 0, (cudaStream_t)stream>>>(d_match_len, d_arrival, d_waiting, nq, kk, d_out,
                                                                            g_topk_scratch[dev]);
    CK(cudaGetLastError());
    return RT_OK;
}

rt_status klpm_select_noalloc(const int32_t* d_match_len, const int64_t* d_arrival, const uint8_t* d_waiting, int32_t nq,
                              int64_t pick_counter, const klpm_params* params, int32_t* d_pick, void* stream) {
    if (!params_ok(params) || nq < 0 || !d_pick || pick_counter < 0 ||
        (nq > 0 && (!d_match_len || !d_arrival || !d_waiting))) return RT_ERR_INVALID;
    if (nq > KLPM_SELECT_NOALLOC_MAX_QUERIES) {
        fprintf(stderr, "klpm_select_noalloc: nq = %d is above the fixed-scratch limit of %d queries; "
                        "use klpm_select for larger queues\n", nq, KLPM_SELECT_NOALLOC_MAX_QUERIES);
        return RT_ERR_TOO_LARGE;
    }
    int dev = 0;
    CK(cudaGetDevice(&dev));
    if (dev < 0 || dev >= 64) return RT_ERR_INVALID;
    if (!g_select_static_addr[dev]) {
        // In host code the array's name only stands for the symbol; the kernel needs its device address.
        StaticSelectScratch* p = nullptr;
        CK(cudaGetSymbolAddress((void**)&p, g_select_static));
        if (!p) return RT_ERR_CUDA;
        g_select_static_addr[dev] = p;
    }
    StaticSelectScratch* sc = g_select_static_addr[dev];
    cudaStream_t s = (cudaStream_t)stream;
    // the arrival counter must start at zero whatever an earlier call left behind
    CK(cudaMemsetAsync(&sc->ticket, 0, sizeof(unsigned int), s));
    const bool fcfs_turn = params->policy == KLPM_POLICY_FCFS ||
                           (params->policy == KLPM_POLICY_KLPM && pick_counter % params->k == 0);
    long long blocks = ((long long)nq + 2047) / 2048;
    if (blocks < 1) blocks = 1;
    if (blocks > KLPM_SELECT_NOALLOC_BLOCKS) blocks = KLPM_SELECT_NOALLOC_BLOCKS;
    if (fcfs_turn) select_static_kernel<false><<<(unsigned)blocks, 512, 0, s>>>(d_match_len, d_arrival, d_waiting, nq, d_pick, sc);
    else select_static_kernel<true><<<(unsigned)blocks, 512, 0, s>>>(d_match_len, d_arrival, d_waiting, nq, d_pick, sc);
    CK(cudaGetLastError());
    return RT_OK;
}

static rt_status run_impl(rt_tree* tree, const int32_t* d_q_tokens, const int64_t* d_q_offsets, const int64_t* d_arrival,
                          int32_t n, const klpm_params* params, const int64_t* d_tie_priority, int32_t score_mode,
                          const klpm_match_state* d_match_state, int32_t* d_order, int32_t* d_uncached, int64_t* d_ttft,
                          int64_t* d_completion, const int32_t* d_fixed, int32_t n_fixed, void* stream);

rt_status klpm_replay(rt_tree* tree, const int32_t* d_order, int32_t n_order, const int32_t* d_q_tokens,
                      const int64_t* d_q_offsets, const int64_t* d_arrival, int32_t n_queries, const klpm_params* params,
                      int32_t* d_uncached, int64_t* d_ttft, int64_t* d_completion, void* stream) {
    if (!tree || !params_ok(params) || n_order < 0 || n_queries < 0 ||
        (n_order > 0 && (!d_order || !d_q_tokens || !d_q_offsets || !d_arrival || !d_uncached || !d_ttft))) return RT_ERR_INVALID;
    if (n_order == 0) return RT_OK;
    // The same loop as klpm_run with the order given instead of picked (every query's match state is kept, a processed
    // prompt re-matches its group only, the tree is written once at the end).  The debug setting run_one_by_one keeps
    // the plain form: one CTA that walks, charges and stores one prompt after the other on the tree itself.
    if (!g_knobs.run_one_by_one && n_queries > 0)
        return run_impl(tree, d_q_tokens, d_q_offsets, d_arrival, n_queries, params, nullptr, 0, nullptr, nullptr, d_uncached, d_ttft,
                        d_completion, d_order, n_order, stream);
    tree->version++;
    SeqArgs a;
    memset(&a, 0, sizeof(a));
    a.tok = d_q_tokens; a.off = d_q_offsets; a.arrival = d_arrival; a.order = d_order; a.n = n_order; a.n_queries = n_queries;
    a.c_num = params->c_num; a.c_den = params->c_den; a.start_tick = params->start_tick;
    a.uncached = d_uncached; a.ttft = d_ttft; a.completion = d_completion;
    tree->last_stream = (cudaStream_t)stream;
    sequential_kernel<<<1, 1024, 0, (cudaStream_t)stream>>>(tree->dev, a);
    CK(cudaGetLastError());
    return RT_OK;
}

rt_status klpm_batch_times(const int32_t* d_order, int32_t n_order, const int64_t* d_arrival, const int64_t* d_completion,
                           int32_t n_queries, int32_t batch_size, int64_t* d_ttft_b, int64_t* d_completion_b,
                           int32_t* d_n_skipped, void* stream) {
    if (n_order < 0 || n_queries < 0 || batch_size < 1 ||
        (n_order > 0 && (!d_order || !d_arrival || !d_completion || !d_ttft_b || !d_completion_b))) return RT_ERR_INVALID;
    if (d_n_skipped) CK(cudaMemsetAsync(d_n_skipped, 0, sizeof(int32_t), (cudaStream_t)stream));
    if (n_order == 0) return RT_OK;
    batch_times_kernel<<<(unsigned)((n_order + 255) / 256), 256, 0, (cudaStream_t)stream>>>(d_order, n_order, d_arrival, d_completion,
                                                                                           n_queries, batch_size, d_ttft_b,
                                                                                           d_completion_b, d_n_skipped);
    CK(cudaGetLastError());
    return RT_OK;
}

// klpm_run_ex, and klpm_replay when d_fixed (a processing order of n_fixed entries) is given: then d_order is null,
// no decision is taken by a policy, and only the prompts of the order are charged and stored.
static rt_status run_impl(rt_tree* tree, const int32_t* d_q_tokens, const int64_t* d_q_offsets, const int64_t* d_arrival,
                          int32_t n, const klpm_params* params, const int64_t* d_tie_priority, int32_t score_mode,
                          const klpm_match_state* d_match_state, int32_t* d_order, int32_t* d_uncached, int64_t* d_ttft,
                          int64_t* d_completion, const int32_t* d_fixed, int32_t n_fixed, void* stream) {
    if (!tree || !params_ok(params) || n < 0 || score_mode < 0 || score_mode > 1 ||
        (n > 0 && (!d_q_tokens || !d_q_offsets || !d_arrival || (!d_order && !d_fixed) || !d_uncached || !d_ttft))) return RT_ERR_INVALID;
    if (n == 0) return RT_OK;
    // records of a batched match are only good for the queries they were written for and the tree as it was then
    if (d_match_state && (tree->ms_state != (const void*)d_match_state || tree->ms_n != n || tree->ms_tok != (const void*)d_q_tokens ||
                          tree->ms_off != (const void*)d_q_offsets || tree->ms_version != tree->version)) return RT_ERR_INVALID;
    cudaStream_t s = (cudaStream_t)stream;
    tree->last_stream = s;
    tree->version++;
    rt_status st = ensure_run_scratch(tree, n);
    if (st) return st;
    long long np2 = 1;
    while (np2 < n) np2 <<= 1;
    // A tree without a budget takes the grouped loop (unless the debug setting run_one_by_one is on).
    const bool grouped = !g_knobs.run_one_by_one;
    const bool lru = tree->cfg.budget_tokens > 0;
    // slots = queries ordered by (arrival, index); for a given order, the queries in index order
    if (d_fixed) {
        replay_slots_kernel<<<(unsigned)((n + 255) / 256), 256, 0, s>>>(d_arrival, n, tree->run_key, tree->run_ord);
        CK(cudaGetLastError());
    } else {
        unsigned blocks = (unsigned)((np2 + 255) / 256);
        rank_init_kernel<<<blocks, 256, 0, s>>>(d_arrival, n, np2, tree->run_key, tree->run_ord);
        sort_pairs(tree->run_key, tree->run_ord, np2, s);
        slot_arrays_kernel<<<(unsigned)((n + 255) / 256), 256, 0, s>>>(tree->run_ord, d_q_offsets, n, tree->run_soff, tree->run_slen);
        if (score_mode == 1) hit_rate_guard_kernel<<<(unsigned)((n + 255) / 256), 256, 0, s>>>(d_q_offsets, n, tree->dev.st);
        if (d_tie_priority) {        // rank of every slot by (priority, slot)
            prio_init_kernel<<<blocks, 256, 0, s>>>(d_tie_priority, tree->run_ord, n, np2, tree->run_pkey, tree->run_pinv);
            sort_pairs(tree->run_pkey, tree->run_pinv, np2, s);
            prio_rank_kernel<<<(unsigned)((n + 255) / 256), 256, 0, s>>>(tree->run_pinv, n, tree->run_prank);
        }
        CK(cudaGetLastError());
    }
    if (grouped) {
        FastArgs f;
        memset(&f, 0, sizeof(f));
        st = ensure_fast_scratch(tree, n);
        if (st) return st;
        st = ensure_bulk_scratch(tree, d_fixed && n_fixed > n ? n_fixed : n);
        if (st) return st;
        if (d_fixed) {
            // which entries of the order will be processed: those before the first that is not a query or comes twice
            if (!tree->replay_info && (st = dalloc(&tree->replay_info, 1))) return st;
            const unsigned fb = (unsigned)((n_fixed + 255) / 256);
            bulk_fill_kernel<<<(unsigned)((n + 255) / 256), 256, 0, s>>>(tree->bulk_pm, n, 0x7fffffff);
            bulk_fill_kernel<<<1, 1, 0, s>>>(&tree->replay_info->n_valid, 1, n_fixed);
            replay_first_kernel<<<fb, 256, 0, s>>>(d_fixed, n_fixed, n, tree->bulk_pm);
            replay_check_kernel<<<fb, 256, 0, s>>>(d_fixed, n_fixed, n, d_q_offsets, tree->bulk_pm, tree->replay_info, tree->dev.st);
            f.fixed = d_fixed; f.n_fixed = &tree->replay_info->n_valid;
        }
        if (lru) {
            if (!tree->lru_parked && (st = dalloc(&tree->lru_parked, tree->dev.max_nodes))) return st;
            if (!tree->lru_info && (st = dalloc(&tree->lru_info, 1))) return st;
            if (n > tree->lru_hintc_cap) {
                cudaFree(tree->lru_hintc);
                tree->lru_hintc = nullptr; tree->lru_hintc_cap = 0;
                if ((st = dalloc(&tree->lru_hintc, n))) return st;
                tree->lru_hintc_cap = n;
            }
            f.hintc = tree->lru_hintc;
            if (!tree->lru_leaf_run && (st = dalloc(&tree->lru_leaf_run, tree->dev.max_nodes))) return st;
            f.leaf_run = tree->lru_leaf_run;
            f.pk = tree->fast_lk; f.pi = tree->fast_ls;      // (the key list of list mode is not used on these trees)
            CK(cudaMemsetAsync(tree->lru_leaf_run, 0xff, (size_t)tree->dev.max_nodes * sizeof(int2), s));
            f.lru = 1; f.T = tree->dev; f.parked = tree->lru_parked; f.skip = &tree->lru_info->skip;
            f.mem_cap = (int32_t)(tree->fast_mem_cap < 0x7fffffffLL ? tree->fast_mem_cap : 0x7fffffffLL);
            // all or nothing: is there room for whatever the loop can leave behind?
            CK(cudaMemsetAsync(tree->lru_info, 0, sizeof(LruInfo), s));
            CK(cudaMemsetAsync(tree->lru_parked, 0, (size_t)tree->dev.max_nodes * sizeof(int32_t), s));
            if (d_fixed) lru_sum_order_kernel<<<(unsigned)((n_fixed + 255) / 256), 256, 0, s>>>(d_q_offsets, d_fixed, n_fixed, n, tree->lru_info);
            else lru_sum_kernel<<<(unsigned)((n + 255) / 256), 256, 0, s>>>(d_q_offsets, n, tree->lru_info);
            lru_check_kernel<<<1, 1, 0, s>>>(tree->dev, d_fixed ? n_fixed : n, tree->lru_info);
        }
        f.tok = d_q_tokens; f.n = n; f.policy = params->policy; f.k = params->k; f.score_mode = score_mode;
        f.c_num = params->c_num; f.c_den = params->c_den; f.start_tick = params->start_tick;
        f.order = d_order; f.uncached = d_uncached; f.ttft = d_ttft; f.completion = d_completion;
        f.dyn = tree->fast_dyn; f.stat = tree->fast_stat; f.key = tree->fast_key_arr; f.mem = tree->fast_mem;
        f.pinv = d_tie_priority ? tree->run_pinv : nullptr;
        f.gh = tree->fast_gh; f.gidx = tree->fast_gidx; f.done = tree->fast_done;
        f.arrival = d_arrival; f.post = tree->fast_post;
        f.vbase = tree->dev.max_pool + 16;
        f.st = tree->dev.st;
        // Every query is matched once against the tree as it stands: by the caller's batched match if it kept the
        // records (rt_match_batch_ex), by the same kernel here otherwise.
        const MatchState* state = reinterpret_cast<const MatchState*>(d_match_state);
        unsigned long long tag = tree->ms_tag;
        if (!state) {
            if (n > tree->own_state_cap) {
                cudaFree(tree->own_state);
                tree->own_state = nullptr; tree->own_state_cap = 0;
                if ((st = dalloc(&tree->own_state, n))) return st;
                tree->own_state_cap = n;
            }
            tag = ++g_match_tag;
            st = launch_match(tree, d_q_tokens, d_q_offsets, n, nullptr, nullptr, nullptr, tree->own_state, tag, s);
            if (st) return st;
            state = tree->own_state;
        }
        fast_stat_kernel<<<(unsigned)((n + 255) / 256), 256, 0, s>>>(tree->run_ord, tree->run_key, d_q_offsets,
                                                                     d_tie_priority ? tree->run_prank : nullptr, n, f.stat);
        fast_state_kernel<<<(unsigned)((np2 + 255) / 256), 256, 0, s>>>(f, state, tag, np2);
        CK(cudaGetLastError());
        // Leaf blocks of 32 slots while at most 8,192 of them are needed, larger ones beyond (queues above 262,144).
        // Two debug settings shrink the limits so that small queues can exercise the large-queue layout:
        // fast_max_blocks (leaf blocks) and fast_smem_kb (shared memory the loop may use).
        long long max_blocks = 8192;
        size_t smem_max = 224 * 1024;
        if (g_knobs.fast_max_blocks >= 1 && g_knobs.fast_max_blocks < max_blocks) max_blocks = g_knobs.fast_max_blocks;
        if (g_knobs.fast_smem_kb >= 1 && (size_t)g_knobs.fast_smem_kb * 1024 < smem_max) smem_max = (size_t)g_knobs.fast_smem_kb * 1024;
        int lbs = 5;
        while ((((long long)n + (1LL << lbs) - 1) >> lbs) > max_blocks) ++lbs;
        f.lb_shift = lbs;
        f.nb = (int32_t)(((long long)n + (1LL << lbs) - 1) >> lbs);
        const long long nb1p = (f.nb + 31) & ~31, n2p = ((nb1p >> 5) + 31) & ~31;
        const long long nwords = ((long long)n + 31) >> 5;
        size_t smem = (size_t)(nb1p + n2p + 32) * 8 + (size_t)KLPM_FAST_SORT_CAP * 12;
        f.done_in_smem = smem + (size_t)nwords * 4 <= smem_max ? 1 : 0;
        if (f.done_in_smem) smem += (size_t)nwords * 4;
        // list mode (trees without a budget) needs two more bitmaps: in shared memory while they fit, in global memory beyond
        f.list_mode = (lru || d_fixed) ? 0 : 1;
        f.bits_in_smem = (f.list_mode && f.done_in_smem && smem + (size_t)nwords * 8 <= smem_max) ? 1 : 0;
        if (f.bits_in_smem) smem += (size_t)nwords * 8;
        f.gbits = tree->fast_done + (np2 / 32 + 32);
        f.gskip = tree->fast_done + 2 * (np2 / 32 + 32);
        const unsigned nblk = (unsigned)((n + 255) / 256), pblk = (unsigned)((np2 + 255) / 256);
        CK(cudaMemsetAsync(f.done, 0, (size_t)(3 * (np2 / 32 + 32)) * sizeof(unsigned int), s));
        // groups: queries whose match ends at the same position and continues with the same token
        sort_pairs(f.gh, f.gidx, np2, s);
        fast_group_kernel<<<nblk, 256, 0, s>>>(f);
        if (lru) {                   // per node of the tree: the slots parked in it as the loop starts
            sort_pairs(f.pk, f.pi, np2, s);
            lru_parklist_kernel<<<nblk, 256, 0, s>>>(f);
        }
        if (f.list_mode) {           // all keys, largest first
            f.lk = tree->fast_lk; f.ls = tree->fast_ls;
            fast_list_kernel<<<pblk, 256, 0, s>>>(f.key, n, np2, tree->fast_lk, tree->fast_ls);
            sort_pairs(tree->fast_lk, tree->fast_ls, np2, s);
        }
        CK(cudaGetLastError());
        if (f.done_in_smem && (f.bits_in_smem || !f.list_mode)) {
            CK(cudaFuncSetAttribute(fast_run_kernel<false>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem));
            fast_run_kernel<false><<<1, KLPM_FAST_THREADS, smem, s>>>(f);
        } else {
            CK(cudaFuncSetAttribute(fast_run_kernel<true>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem));
            fast_run_kernel<true><<<1, KLPM_FAST_THREADS, smem, s>>>(f);
        }
        if (f.list_mode) {           // the decisions made in list mode are charged here (none if list mode never began)
            const int32_t ipt = (int32_t)(((long long)n + 1024LL * KLPM_CHARGE_THREADS - 1) / (1024LL * KLPM_CHARGE_THREADS));
            const int32_t per_block = KLPM_CHARGE_THREADS * ipt;
            const int32_t cblocks = (n + per_block - 1) / per_block;                          // at most 1,024
            charge_cost_kernel<<<cblocks, KLPM_CHARGE_THREADS, 0, s>>>(f, tree->fast_gh, tree->fast_bsum, ipt);
            charge_scan_kernel<<<1, 1024, 0, s>>>(f, tree->fast_bsum, cblocks);
            charge_apply_kernel<<<cblocks, KLPM_CHARGE_THREADS, 0, s>>>(f, tree->fast_gh, tree->fast_bsum, ipt);
        }
        CK(cudaGetLastError());
        tree->run_path = 2;
        if (lru) {
            // the nodes that are alive after the loop get their tokens, and the child table is written afresh
            const TreeDev& d = tree->dev;
            lru_tokens_kernel<<<(unsigned)tree->num_sms * 8, 256, 0, s>>>(d, d_fixed ? d_fixed : d_order, d_q_tokens, d_q_offsets, f.vbase, tree->lru_info);
            table_clear_kernel<<<(unsigned)tree->num_sms * 8, 256, 0, s>>>(d, tree->lru_info);
            lru_table_kernel<<<(unsigned)((d.max_nodes + 255) / 256), 256, 0, s>>>(d, f.vbase, tree->lru_info);
            CK(cudaGetLastError());
            return RT_OK;
        }
        // The processed prompts enter the tree together (the logical clock advances by n).  The loop itself needs
        // no room in the tree; if the tree cannot hold the queue the insertion says so through the status word.
        if (d_fixed) {               // only the prompts of the order, and the clock advances by as many as were processed
            replay_list_kernel<<<(unsigned)((n_fixed + 255) / 256), 256, 0, s>>>(d_fixed, n_fixed, tree->replay_info, tree->bulk_pend_a);
            return bulk_insert(tree, d_q_tokens, d_q_offsets, n_fixed, s, state, tag, true, &tree->replay_info->n_valid);
        }
        return bulk_insert(tree, d_q_tokens, d_q_offsets, n, s, state, tag);
    }
    if (d_fixed) return RT_ERR_INVALID;       // (klpm_replay takes its sequential kernel instead of this loop)
    RunBcast bc0;
    memset(&bc0, 0, sizeof(bc0));
    bc0.now = params->start_tick;
    CK(cudaMemcpyAsync(tree->run_bc, &bc0, sizeof(bc0), cudaMemcpyHostToDevice, s));
    CK(cudaMemsetAsync(tree->run_sy, 0, sizeof(RunSync), s));
    RunArgs a;
    memset(&a, 0, sizeof(a));
    a.tok = d_q_tokens; a.off = d_q_offsets; a.arrival = d_arrival; a.n = n;
    a.policy = params->policy; a.k = params->k; a.c_num = params->c_num; a.c_den = params->c_den; a.start_tick = params->start_tick;
    a.order = d_order; a.uncached = d_uncached; a.ttft = d_ttft; a.completion = d_completion;
    a.soff = tree->run_soff; a.slen = tree->run_slen; a.ntok = tree->run_ntok;
    a.prank = d_tie_priority ? tree->run_prank : nullptr; a.pinv = d_tie_priority ? tree->run_pinv : nullptr;
    a.score_mode = score_mode;
    a.ord = tree->run_ord; a.sorted_t = tree->run_key; a.m = tree->run_m; a.hint = tree->run_hint; a.pos = tree->run_pos;
    a.partial = tree->run_partial; a.bc = tree->run_bc; a.sy = tree->run_sy;
    a.wait_limit_ns = g_knobs.wait_limit_ns;
    const int threads = KLPM_RUN_THREADS;
    int per_sm = 0;
    CK(cudaOccupancyMaxActiveBlocksPerMultiprocessor(&per_sm, run_kernel, threads, 0));
    if (per_sm < 1) return RT_ERR_CUDA;
    // one sequencer CTA plus scanners; small queues are handled by the sequencer alone
    long long blocks = 1;
    if (n > threads * 8) blocks = 1 + ((long long)n + threads * KLPM_RUN_SPT - 1) / (threads * KLPM_RUN_SPT);
    if (blocks > tree->num_sms) blocks = tree->num_sms;
    void* kargs[] = {(void*)&tree->dev, (void*)&a};
    CK(cudaLaunchCooperativeKernel((void*)run_kernel, dim3((unsigned)blocks), dim3(threads), kargs, 0, s));
    tree->run_path = 1;
    return RT_OK;
}

rt_status klpm_run_last_only_batch(const int32_t* d_tokens, const int64_t* d_offsets, const int64_t* d_arrival,
                                   const int64_t* d_tie_priority, const int32_t* d_queue_offsets, int32_t n_queues,
                                   const klpm_params* params, int32_t* d_order, int32_t* d_uncached, int64_t* d_ttft,
                                   int64_t* d_completion, int32_t* d_n_skipped, void* stream) {
    if (!params_ok(params) || n_queues < 0 ||
        (n_queues > 0 && (!d_tokens || !d_offsets || !d_arrival || !d_queue_offsets || !d_order || !d_uncached || !d_ttft)))
        return RT_ERR_INVALID;
    cudaStream_t s = (cudaStream_t)stream;
    if (d_n_skipped) CK(cudaMemsetAsync(d_n_skipped, 0, sizeof(int32_t), s));
    if (n_queues == 0) return RT_OK;
    LastOnlyArgs a;
    a.tok = d_tokens; a.off = d_offsets; a.arrival = d_arrival; a.prio = d_tie_priority; a.qoff = d_queue_offsets;
    a.n_queues = n_queues; a.policy = params->policy; a.k = params->k;
    a.c_num = params->c_num; a.c_den = params->c_den; a.start_tick = params->start_tick;
    a.order = d_order; a.uncached = d_uncached; a.ttft = d_ttft; a.completion = d_completion; a.n_skipped = d_n_skipped;
    const unsigned blocks = (unsigned)(((long long)n_queues + KLPM_LAST_ONLY_WARPS - 1) / KLPM_LAST_ONLY_WARPS);
    last_only_batch_kernel<<<blocks, 32 * KLPM_LAST_ONLY_WARPS, 0, s>>>(a);
    CK(cudaGetLastError());
    return RT_OK;
}

rt_status klpm_run_ex(rt_tree* tree, const int32_t* d_q_tokens, const int64_t* d_q_offsets, const int64_t* d_arrival,
                      int32_t n, const klpm_params* params, const int64_t* d_tie_priority, int32_t score_mode,
                      const klpm_match_state* d_match_state, int32_t* d_order, int32_t* d_uncached, int64_t* d_ttft,
                      int64_t* d_completion, void* stream) {
    if (n > 0 && !d_order) return RT_ERR_INVALID;
    return run_impl(tree, d_q_tokens, d_q_offsets, d_arrival, n, params, d_tie_priority, score_mode, d_match_state, d_order,
                    d_uncached, d_ttft, d_completion, nullptr, 0, stream);
}

int32_t klpm_run_path(const rt_tree* tree) { return tree ? tree->run_path : 0; }

rt_status rt_debug_counters(rt_tree* tree, int64_t* out16) {
    if (!tree || !out16) return RT_ERR_INVALID;
    memset(out16, 0, 16 * sizeof(int64_t));
    if (!tree->fast_post) return RT_OK;
    CK(cudaStreamSynchronize(tree->last_stream));
    FastPost h;
    CK(cudaMemcpy(&h, tree->fast_post, sizeof(h), cudaMemcpyDeviceToHost));
    for (int i = 0; i < 16; ++i) out16[i] = h.counters[i];
    return RT_OK;
}

rt_status klpm_debug_set(const char* name, int64_t value) {
    if (!name) return RT_ERR_INVALID;
    const DebugKnobs defaults = {0, 0, 0, KLPM_WAIT_LIMIT_NS};
    if (!strcmp(name, "run_one_by_one")) g_knobs.run_one_by_one = value < 0 ? defaults.run_one_by_one : (value != 0);
    else if (!strcmp(name, "fast_max_blocks")) g_knobs.fast_max_blocks = value < 0 ? defaults.fast_max_blocks : value;
    else if (!strcmp(name, "fast_smem_kb")) g_knobs.fast_smem_kb = value < 0 ? defaults.fast_smem_kb : value;
    else if (!strcmp(name, "wait_limit_ns")) g_knobs.wait_limit_ns = value < 0 ? defaults.wait_limit_ns : value;
    else return RT_ERR_INVALID;
    return RT_OK;
}

rt_status klpm_run(rt_tree* tree, const int32_t* d_q_tokens, const int64_t* d_q_offsets, const int64_t* d_arrival,
                   int32_t n, const klpm_params* params, int32_t* d_order, int32_t* d_uncached, int64_t* d_ttft,
                   int64_t* d_completion, void* stream) {
    return klpm_run_ex(tree, d_q_tokens, d_q_offsets, d_arrival, n, params, nullptr, 0, nullptr, d_order, d_uncached, d_ttft,
                       d_completion, stream);
}

}  // extern "C"
