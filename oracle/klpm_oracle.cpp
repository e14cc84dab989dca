// CPU oracle for the k-LPM scheduling path.  TEST INFRASTRUCTURE ONLY.
//
// A plain, slow, single-purpose restatement of what the paper defines, used to
// check the CUDA library and to give a CPU baseline.  It shares no code with
// the CUDA path.  Only the test-suite, the smoke check and the benchmark's CPU
// baseline may load it; the product never does.
//
// What it computes, and where the paper defines it:
//   overlap(x, y)      length of the maximal common prefix       (Section 1.3, Notation)
//   query stream       prompts x_i with arrival ticks t_i        (Definition 1)
//   completion times   R(j_k) = max{R(j_{k-1}), t_{j_k}}
//                        + (1 + c_attn |x|)(|x| - overlap)        (Definition 2)
//   cache              LAST_ONLY: only the previously processed prompt is cached
//                        (Definition 2 and Section 2.1);
//                      TREE: a radix tree of every processed prompt with LRU
//                        eviction under a fixed token budget (Section 1, RadixAttention)
//   policies           FCFS, LPM (Section 1) and k-LPM (Algorithm 1)
//
// Readings taken where the paper is silent:
//   * Algorithm 1 is followed as printed: one oldest-first pick, then k-1
//     longest-match picks; the pick counter never resets (idle periods included).
//   * "prefix cache hit rate" is the absolute match length in tokens; the other reading
//     (score_mode 1) is the rational m / |x|, compared exactly by cross-multiplication.
//   * ties go to the earliest arrival, then to the lower index.
//   * processing starts at start_tick with the given cache; the recurrence of
//     Definition 2 is applied to the first processed query too.
//   * c_attn is the rational c_num/c_den; times are in units of 1/c_den tick, so
//     cost = (c_den + c_num |x|)(|x| - m) is an exact integer.
//   * LRU: whole leaves are evicted, smallest last_access first; last_access of a
//     node is the logical clock of the last processed prompt whose path covers
//     it; the path of the prompt being processed is stamped before eviction
//     and is therefore never evicted; single-child nodes are not merged.
//   * processing x with match length m puts node boundaries at depth m and |x|.
//
// Parity pins (the CPU test-suite): brute-force LCP against every cached
// prompt; the printed toy example; k=1 -> FCFS and k>n -> LPM limits; the
// closed forms of the proof of Theorem 2; exhaustive permutation search;
// the NP-hardness gadget worked by hand.  The LRU reading has no value in the
// paper to pin against ("parity unpinned" by the paper); it is pinned against
// an independent brute-force set-of-strings model in oracle/definition.py.
#include <algorithm>
#include <cstdint>
#include <cstring>
#include <map>
#include <set>
#include <thread>
#include <vector>

namespace {

typedef int32_t tok_t;

// Section 1.3: length of the maximal prefix overlap of x and y.
int64_t overlap(const tok_t* x, int64_t nx, const tok_t* y, int64_t ny) {
    int64_t n = nx < ny ? nx : ny, i = 0;
    while (i < n && x[i] == y[i]) ++i;
    return i;
}

struct Node {
    Node* parent = nullptr;
    int64_t id = 0;
    int32_t depth_start = 0;                 // tokens on the path above this node
    std::vector<tok_t> span;                 // the edge label leading into this node
    std::map<tok_t, Node*> child;            // keyed by the first token of the child's span
    int64_t last_access = 0;
    bool is_leaf() const { return child.empty(); }
};

struct Tree {
    Node* root;
    int64_t budget;        // tokens, 0 = unbounded
    int64_t tokens = 0;    // tokens held by live nodes
    int64_t clock = 0;     // logical clock: +1 per processed prompt
    int64_t n_nodes = 0;   // live nodes, root excluded
    int64_t next_id = 1;
    int64_t evictions = 0;
    bool indexed;          // keep an ordered index of leaves (same answer as the linear scan, faster)
    std::set<std::pair<int64_t, Node*>> leaves;   // (last_access, node) of every live leaf, if indexed
    std::vector<Node*> all;                        // every live node, if not indexed

    Tree(int64_t b, bool idx) : budget(b), indexed(idx) { root = new Node(); }
    ~Tree() { destroy(root); }
    static void destroy(Node* n) {
        for (auto& kv : n->child) destroy(kv.second);
        delete n;
    }
};

struct Pos { Node* node; int32_t off; int32_t m; };   // m tokens matched; `off` of them inside node's span

// Longest prefix of x that lies on a root path; partial edges count token by token.
Pos walk(const Tree& t, const tok_t* x, int64_t nx) {
    Node* cur = t.root;
    int32_t m = 0;
    for (;;) {
        if (m == nx) return Pos{cur, (int32_t)cur->span.size(), m};
        auto it = cur->child.find(x[m]);
        if (it == cur->child.end()) return Pos{cur, (int32_t)cur->span.size(), m};
        Node* c = it->second;
        int64_t o = overlap(x + m, nx - m, c->span.data(), (int64_t)c->span.size());
        m += (int32_t)o;
        if (o < (int64_t)c->span.size()) return Pos{c, (int32_t)o, m};
        cur = c;
    }
}

void leaf_index_remove(Tree& t, Node* n) { if (t.indexed) t.leaves.erase({n->last_access, n}); }
void leaf_index_add(Tree& t, Node* n) { if (t.indexed && n != t.root && n->is_leaf()) t.leaves.insert({n->last_access, n}); }

void stamp(Tree& t, Node* n, int64_t clock) {
    if (n == t.root) return;
    if (n->is_leaf()) leaf_index_remove(t, n);
    n->last_access = clock;
    leaf_index_add(t, n);
}

// Put a node boundary `off` tokens into node c's span (0 < off < |span|): a new
// upper node takes span[0:off) and keeps c's place under c's parent; c keeps the rest.
Node* split(Tree& t, Node* c, int32_t off) {
    Node* up = new Node();
    up->id = t.next_id++;
    up->parent = c->parent;
    up->depth_start = c->depth_start;
    up->span.assign(c->span.begin(), c->span.begin() + off);
    up->last_access = c->last_access;
    c->parent->child[up->span[0]] = up;
    c->span.erase(c->span.begin(), c->span.begin() + off);
    c->depth_start += off;
    c->parent = up;
    up->child[c->span[0]] = c;
    t.n_nodes++;
    if (!t.indexed) t.all.push_back(up);
    return up;
}

// The live leaf with the smallest last_access, or null.
Node* oldest_leaf(Tree& t) {
    if (t.indexed) return t.leaves.empty() ? nullptr : t.leaves.begin()->second;
    Node* best = nullptr;
    for (Node* n : t.all)
        if (n->is_leaf() && (!best || n->last_access < best->last_access)) best = n;
    return best;
}

void evict(Tree& t, Node* leaf) {
    Node* p = leaf->parent;
    leaf_index_remove(t, leaf);
    p->child.erase(leaf->span[0]);
    t.tokens -= (int64_t)leaf->span.size();
    t.n_nodes--;
    t.evictions++;
    if (!t.indexed) t.all.erase(std::find(t.all.begin(), t.all.end(), leaf));
    delete leaf;
    leaf_index_add(t, p);     // the parent may have become a leaf
}

// Process prompt x (Section 1: its KV cache is stored in the tree).  Returns the number of
// uncached tokens |x| - m, or -1 if the budget cannot hold the prompt.
int64_t process(Tree& t, const tok_t* x, int64_t nx, bool* evicted_any) {
    t.clock++;
    Pos p = walk(t, x, nx);
    Node* end = p.node;
    if (p.node != t.root && p.off < (int32_t)p.node->span.size()) end = split(t, p.node, p.off);
    for (Node* a = end; a != t.root; a = a->parent) stamp(t, a, t.clock);
    int64_t unc = nx - p.m;
    if (t.budget > 0) {
        while (t.tokens + unc > t.budget) {
            Node* v = oldest_leaf(t);
            if (!v || v->last_access >= t.clock) return -1;
            evict(t, v);
            if (evicted_any) *evicted_any = true;
        }
    }
    if (unc > 0) {
        Node* leaf = new Node();
        leaf->id = t.next_id++;
        leaf->parent = end;
        leaf->depth_start = p.m;
        leaf->span.assign(x + p.m, x + nx);
        leaf->last_access = t.clock;
        if (end != t.root && end->is_leaf()) leaf_index_remove(t, end);
        end->child[leaf->span[0]] = leaf;
        t.tokens += unc;
        t.n_nodes++;
        if (!t.indexed) t.all.push_back(leaf);
        leaf_index_add(t, leaf);
    }
    return unc;
}

enum { POLICY_FCFS = 0, POLICY_LPM = 1, POLICY_KLPM = 2 };
enum { CACHE_LAST_ONLY = 0, CACHE_TREE = 1 };
enum { TIER_REMATCH = 1, TIER_UPDATE = 2 };

struct Stream {
    const tok_t* tok; const int64_t* off; const int64_t* arrival; int32_t n;
    const tok_t* x(int32_t i) const { return tok + off[i]; }
    int64_t len(int32_t i) const { return off[i + 1] - off[i]; }
};

bool earlier(const Stream& s, int32_t a, int32_t b) {      // (t_a, a) < (t_b, b)
    return s.arrival[a] < s.arrival[b] || (s.arrival[a] == s.arrival[b] && a < b);
}

}  // namespace

extern "C" {

int64_t oc_overlap(const tok_t* x, int64_t nx, const tok_t* y, int64_t ny) { return overlap(x, nx, y, ny); }

// Definition-level match: match_len[i] = max(match_len[i], max_y overlap(q_i, y)) over the given cached prompts.
void oc_match_bruteforce(const tok_t* qt, const int64_t* qo, int32_t nq,
                         const tok_t* ct, const int64_t* co, int32_t nc, int32_t* match_len) {
    for (int32_t i = 0; i < nq; ++i)
        for (int32_t j = 0; j < nc; ++j) {
            int64_t o = overlap(qt + qo[i], qo[i + 1] - qo[i], ct + co[j], co[j + 1] - co[j]);
            if (o > match_len[i]) match_len[i] = (int32_t)o;
        }
}

void* oc_tree_new(int64_t budget_tokens, int32_t indexed) { return new Tree(budget_tokens, indexed != 0); }
void oc_tree_free(void* t) { delete (Tree*)t; }

void oc_tree_stats(void* tp, int64_t* n_nodes, int64_t* tokens, int64_t* clock, int64_t* evictions) {
    Tree& t = *(Tree*)tp;
    if (n_nodes) *n_nodes = t.n_nodes;
    if (tokens) *tokens = t.tokens;
    if (clock) *clock = t.clock;
    if (evictions) *evictions = t.evictions;
}

// Process n prompts one after the other.  new_tokens[i] (nullable) = |x_i| - match at its own insertion.
int32_t oc_tree_insert(void* tp, const tok_t* tok, const int64_t* off, int32_t n, int32_t* new_tokens) {
    Tree& t = *(Tree*)tp;
    for (int32_t i = 0; i < n; ++i) {
        int64_t unc = process(t, tok + off[i], off[i + 1] - off[i], nullptr);
        if (unc < 0) return -3;
        if (new_tokens) new_tokens[i] = (int32_t)unc;
    }
    return 0;
}

// match_len[i] = longest prefix of query i on a root path of the tree (read-only).
void oc_tree_match(void* tp, const tok_t* tok, const int64_t* off, int32_t n, int32_t* match_len, int32_t threads) {
    const Tree& t = *(Tree*)tp;
    if (threads < 1) threads = 1;
    std::vector<std::thread> pool;
    for (int32_t w = 0; w < threads; ++w) {
        int32_t lo = (int32_t)((int64_t)n * w / threads), hi = (int32_t)((int64_t)n * (w + 1) / threads);
        auto job = [&t, tok, off, match_len, lo, hi]() {
            for (int32_t i = lo; i < hi; ++i) match_len[i] = walk(t, tok + off[i], off[i + 1] - off[i]).m;
        };
        if (threads == 1) job(); else pool.emplace_back(job);
    }
    for (auto& th : pool) th.join();
}

// The same walk, also reporting where each match ended: term_off[i] = how many tokens of the edge that holds the
// last matched token were matched (0 when nothing matched), term_depth[i] = tokens on the path above that edge.
void oc_tree_match_pos(void* tp, const tok_t* tok, const int64_t* off, int32_t n, int32_t* match_len,
                       int32_t* term_off, int32_t* term_depth) {
    const Tree& t = *(Tree*)tp;
    for (int32_t i = 0; i < n; ++i) {
        Pos p = walk(t, tok + off[i], off[i + 1] - off[i]);
        match_len[i] = p.m;
        term_off[i] = p.off;
        term_depth[i] = p.m - p.off;
    }
}

// Definition 2 along a given processing order.  The cache starts as `tp` holds it (TREE) or empty (LAST_ONLY).
int32_t oc_replay(void* tp, const int32_t* order, int32_t n_order, const tok_t* tok, const int64_t* off,
                  const int64_t* arrival, int32_t n, int64_t c_num, int64_t c_den, int64_t start_tick,
                  int32_t cache_mode, int32_t* uncached, int64_t* ttft, int64_t* completion) {
    Stream s{tok, off, arrival, n};
    Tree* t = (Tree*)tp;
    int64_t now = start_tick;
    int32_t last = -1;
    for (int32_t k = 0; k < n_order; ++k) {
        int32_t j = order[k];
        int64_t len = s.len(j), unc;
        if (cache_mode == CACHE_LAST_ONLY) {
            unc = len - (last < 0 ? 0 : overlap(s.x(j), len, s.x(last), s.len(last)));
            last = j;
        } else {
            unc = process(*t, s.x(j), len, nullptr);
            if (unc < 0) return -3;
        }
        int64_t begin = now > arrival[j] ? now : arrival[j];
        int64_t R = begin + (c_den + c_num * len) * unc;
        if (uncached) uncached[j] = (int32_t)unc;
        if (ttft) ttft[j] = R - arrival[j];
        if (completion) completion[j] = R;
        now = R;
    }
    return 0;
}

// Batch size B (Section 2.1): the processing order is cut into consecutive bins of B queries; a query is
// finished when the last query of its bin is.  completion_b / ttft_b are indexed by query.
void oc_batch_times(const int32_t* order, int32_t n_order, const int64_t* arrival, const int64_t* completion,
                    int32_t B, int64_t* ttft_b, int64_t* completion_b) {
    for (int32_t i = 0; i < n_order; ++i) {
        int32_t last = (i / B + 1) * B - 1;
        if (last > n_order - 1) last = n_order - 1;
        const int64_t R = completion[order[last]];
        completion_b[order[i]] = R;
        ttft_b[order[i]] = R - arrival[order[i]];
    }
}

// One decision of Algorithm 1 as a function of its inputs: among the waiting queries, the oldest one (smallest arrival,
// then index) on an oldest-first turn -- FCFS always, k-LPM when pick_counter is a multiple of k -- and otherwise the
// one with the longest match, ties to the oldest.  Returns its index, or -1 if nobody is waiting.
int32_t oc_select(const int32_t* match_len, const int64_t* arrival, const uint8_t* waiting, int32_t n,
                  int64_t pick_counter, int32_t policy, int32_t k) {
    const bool fcfs_turn = policy == POLICY_FCFS || (policy == POLICY_KLPM && pick_counter % k == 0);
    int32_t j = -1;
    for (int32_t i = 0; i < n; ++i) {
        if (!waiting[i]) continue;
        bool wins = j < 0;
        if (!wins && !fcfs_turn && match_len[i] != match_len[j]) wins = match_len[i] > match_len[j];
        else if (!wins) wins = arrival[i] < arrival[j];      // equal arrivals: the lower index stays
        if (wins) j = i;
    }
    return j;
}

// Algorithm 1 (k-LPM) with its FCFS and LPM limits, run over the whole stream.
// order[c] = index processed at decision c; uncached/ttft/completion are indexed by query.
// Variants of the longest-match pick (both leave the oldest-first picks alone):
//   tie_priority (nullable): among queries with the same score the one with the smallest priority wins, before
//     arrival and index decide.  With priorities drawn at random this is the uniform tie-breaking the paper
//     assumes for LPM (footnote to Theorem 2); the numbers are an input, nothing is drawn here.
//   score_mode 0: score = match length (tokens).  score_mode 1: score = hit rate of the prompt, the rational
//     match / |x| (0 for an empty prompt), compared exactly -- the other reading of "prefix cache hit rate".
int32_t oc_schedule_ex(void* tp, const tok_t* tok, const int64_t* off, const int64_t* arrival, int32_t n,
                       int32_t policy, int32_t k, int64_t c_num, int64_t c_den, int64_t start_tick,
                       int32_t cache_mode, int32_t tier, const int64_t* tie_priority, int32_t score_mode,
                       int32_t* order, int32_t* uncached, int64_t* ttft, int64_t* completion) {
    Stream s{tok, off, arrival, n};
    Tree* t = (Tree*)tp;
    std::vector<char> processed(n, 0), waiting(n, 0);
    std::vector<int32_t> m(n, 0);          // tier 2: current match length of every waiting query
    int32_t last = -1;
    int64_t now = start_tick;

    auto match_now = [&](int32_t i) -> int32_t {
        if (cache_mode == CACHE_LAST_ONLY)
            return last < 0 ? 0 : (int32_t)overlap(s.x(i), s.len(i), s.x(last), s.len(last));
        return walk(*t, s.x(i), s.len(i)).m;
    };

    for (int32_t c = 0; c < n; ++c) {
        // the waiting queue: arrived and not yet processed; idle until the next arrival if empty
        bool any = false;
        for (int32_t i = 0; i < n; ++i) any = any || (!processed[i] && arrival[i] <= now);
        if (!any) {
            int64_t next = -1;
            for (int32_t i = 0; i < n; ++i)
                if (!processed[i] && (next < 0 || arrival[i] < next)) next = arrival[i];
            now = next;
        }
        for (int32_t i = 0; i < n; ++i)
            if (!processed[i] && !waiting[i] && arrival[i] <= now) {
                waiting[i] = 1;
                if (tier == TIER_UPDATE) m[i] = match_now(i);
            }

        bool fcfs_turn = policy == POLICY_FCFS || (policy == POLICY_KLPM && c % k == 0);
        int32_t j = -1;
        if (fcfs_turn) {
            for (int32_t i = 0; i < n; ++i)
                if (waiting[i] && (j < 0 || earlier(s, i, j))) j = i;
        } else {
            int64_t best_num = 0, best_den = 1;     // score of j as a fraction (denominator 1 for match lengths)
            for (int32_t i = 0; i < n; ++i) {
                if (!waiting[i]) continue;
                int32_t mi = tier == TIER_UPDATE ? m[i] : match_now(i);
                if (tier != TIER_UPDATE) m[i] = mi;
                int64_t num = mi, den = 1;
                if (score_mode == 1) { if (s.len(i) > 0) den = s.len(i); else num = 0; }
                // num/den against best_num/best_den, exactly (all four are below 2^31)
                const int64_t lhs = num * best_den, rhs = best_num * den;
                bool wins = j < 0 || lhs > rhs;
                if (!wins && lhs == rhs) {
                    if (tie_priority && tie_priority[i] != tie_priority[j]) wins = tie_priority[i] < tie_priority[j];
                    else wins = earlier(s, i, j);
                }
                if (wins) { j = i; best_num = num; best_den = den; }
            }
        }

        // Definition 2: charge the uncached part of x_j, then x_j enters the cache
        int64_t len = s.len(j), unc;
        bool evicted = false;
        if (cache_mode == CACHE_LAST_ONLY) {
            unc = len - match_now(j);
        } else {
            unc = process(*t, s.x(j), len, &evicted);
            if (unc < 0) return -3;
        }
        int64_t begin = now > arrival[j] ? now : arrival[j];
        int64_t R = begin + (c_den + c_num * len) * unc;
        order[c] = j;
        if (uncached) uncached[j] = (int32_t)unc;
        if (ttft) ttft[j] = R - arrival[j];
        if (completion) completion[j] = R;
        now = R;
        processed[j] = 1;
        waiting[j] = 0;
        int32_t prev_last = last;
        last = j;
        (void)prev_last;

        if (tier == TIER_UPDATE) {
            for (int32_t i = 0; i < n; ++i) {
                if (!waiting[i]) continue;
                if (cache_mode == CACHE_LAST_ONLY || evicted) {
                    m[i] = match_now(i);
                } else {
                    // a prefix-closed cache S plus prompt p matches max(match(q,S), overlap(q,p))
                    int32_t o = (int32_t)overlap(s.x(i), s.len(i), s.x(j), len);
                    if (o > m[i]) m[i] = o;
                }
            }
        }
    }
    return 0;
}

// Algorithm 1 as printed: match length as the score, ties to the earliest arrival.
int32_t oc_schedule(void* tp, const tok_t* tok, const int64_t* off, const int64_t* arrival, int32_t n,
                    int32_t policy, int32_t k, int64_t c_num, int64_t c_den, int64_t start_tick,
                    int32_t cache_mode, int32_t tier,
                    int32_t* order, int32_t* uncached, int64_t* ttft, int64_t* completion) {
    return oc_schedule_ex(tp, tok, off, arrival, n, policy, k, c_num, c_den, start_tick, cache_mode, tier, nullptr, 0,
                          order, uncached, ttft, completion);
}

}  // extern "C"
