// Tri-gram store on the GPU (Eq. 1 counts, Algorithm 2 update, top-k continuation lookup).
//
// Layout: an array of 64-byte buckets.  The first 2^log2_buckets are "home" buckets, found by
// hashing the two-token context (a, b) and probing linearly; a context owns its home bucket and,
// when it has more than six continuations, a chain of overflow buckets taken from a bump
// allocator.  A bucket holds the context key, the index of the next bucket of the chain (0 = none)
// and six (token, count) entries that fill front to back and are never removed.  All contexts'
// continuations are therefore reachable from one hash probe, which is what top-k needs, and an
// update is one probe plus one atomic add.
#include <cmath>
#include <cstdio>
#include <cstring>
#include <new>
#include <vector>

#include "aded_internal.cuh"

namespace aded {

struct TgSlot { int32_t tok; uint32_t cnt; };
struct __align__(64) Bucket {
    unsigned long long key;
    uint32_t next;
    uint32_t pad;
    TgSlot e[6];
};
static_assert(sizeof(Bucket) == 64, "bucket must be 64 bytes");

constexpr unsigned long long TG_EMPTY = ~0ull;
constexpr int TG_MAX_PROBE = 4096;
constexpr uint32_t TG_LOCKED = 0xFFFFFFFFu;   // `next` while its chain is being extended
constexpr int TG_MAX_SPIN = 1 << 20;

struct TgView {
    Bucket* buckets;
    uint32_t n_home_mask;
    uint32_t n_home;
    uint32_t n_over;
    uint32_t* over_used;
    int32_t* status;
    int32_t vocab;
    uint32_t cap;
    uint32_t min_count;
};

__device__ __forceinline__ uint32_t tg_hash(unsigned long long k) {
    k ^= k >> 30; k *= 0xBF58476D1CE4E5B9ull;
    k ^= k >> 27; k *= 0x94D049BB133111EBull;
    k ^= k >> 31;
    return (uint32_t)k;
}

__device__ __forceinline__ unsigned long long tg_key(int a, int b) {
    return ((unsigned long long)(uint32_t)a << 32) | (uint32_t)b;
}

// Home bucket of a context; claims an empty one when `insert`.  Returns -1 if absent / no room.
__device__ __forceinline__ int64_t tg_find_home(const TgView& t, unsigned long long key, bool insert) {
    const uint32_t h = tg_hash(key);
    const int limit = t.n_home < (uint32_t)TG_MAX_PROBE ? (int)t.n_home : TG_MAX_PROBE;
    for (int probe = 0; probe < limit; ++probe) {
        const uint32_t idx = (h + probe) & t.n_home_mask;
        unsigned long long k = *reinterpret_cast<volatile unsigned long long*>(&t.buckets[idx].key);
        if (k == key) return idx;
        if (k == TG_EMPTY) {
            if (!insert) return -1;
            k = atomicCAS(&t.buckets[idx].key, TG_EMPTY, key);
            if (k == TG_EMPTY || k == key) return idx;
        }
    }
    return -1;
}

__global__ void k_tg_init(Bucket* b, size_t n) {
    for (size_t i = blockIdx.x * (size_t)blockDim.x + threadIdx.x; i < n; i += (size_t)gridDim.x * blockDim.x) {
        Bucket z;
        z.key = TG_EMPTY;
        z.next = 0;
        z.pad = 0;
        for (int e = 0; e < 6; ++e) { z.e[e].tok = -1; z.e[e].cnt = 0; }
        b[i] = z;
    }
}

// Raises the count of tri-gram (a, b, c) by `inc` (1 <= inc <= cap), inserting it if absent; counts
// saturate at the cap.  Independent atomic adds: the result does not depend on the thread order.
__device__ __forceinline__ void tg_add(const TgView& t, int a, int b, int c, uint32_t inc) {
    const unsigned long long key = tg_key(a, b);
    int64_t cur = tg_find_home(t, key, true);
    if (cur < 0) { atomicCAS(t.status, 0, (int)ADED_ERR_TABLE_FULL); return; }
    // a chain can never be longer than every overflow bucket plus the home bucket
    for (uint32_t hop = 0; hop <= t.n_over; ++hop) {
        if (!ADED_IN_RANGE(cur >= 0 && (uint64_t)cur < (uint64_t)t.n_home + t.n_over, t.status)) return;
        Bucket* bk = t.buckets + cur;
        for (int e = 0; e < 6; ++e) {
            int32_t have = *reinterpret_cast<volatile int32_t*>(&bk->e[e].tok);
            if (have == -1) have = atomicCAS(&bk->e[e].tok, -1, c) == -1 ? c : *reinterpret_cast<volatile int32_t*>(&bk->e[e].tok);
            if (have == c) {
                if (inc == 1) {
                    // the per-step update: cap <= 2^31 - 1 and at most 2^31 threads add 1 before the minimum below
                    // takes effect, so the 32-bit count cannot wrap
                    const uint32_t old = atomicAdd(&bk->e[e].cnt, 1u);
                    if (old >= t.cap) atomicMin(&bk->e[e].cnt, t.cap);
                } else {
                    // imports add arbitrary counts: saturate in one step, so that two large additions to one
                    // tri-gram cannot carry the count past 2^32 between an add and a later minimum
                    uint32_t seen = *reinterpret_cast<volatile uint32_t*>(&bk->e[e].cnt);
                    for (;;) {
                        const uint32_t want = seen >= t.cap || inc > t.cap - seen ? t.cap : seen + inc;
                        const uint32_t prev = atomicCAS(&bk->e[e].cnt, seen, want);
                        if (prev == seen) break;
                        seen = prev;      // (another thread moved the count; every retry follows a change made by someone else)
                    }
                }
                return;
            }
        }
        // Extend the chain under a one-word lock so that concurrent inserts into a hot context do
        // not each take a bucket: the thread that swings `next` from 0 to TG_LOCKED allocates and
        // publishes the index; the others wait for it, for a bounded number of polls.
        uint32_t nxt = *reinterpret_cast<volatile uint32_t*>(&bk->next);
        if (nxt == 0) {
            const uint32_t prev = atomicCAS(&bk->next, 0u, TG_LOCKED);
            if (prev == 0) {
                const uint32_t fresh = atomicAdd(t.over_used, 1u);
                if (fresh >= t.n_over) {
                    atomicExch(&bk->next, 0u);
                    atomicCAS(t.status, 0, (int)ADED_ERR_TABLE_FULL);
                    return;
                }
                nxt = t.n_home + fresh;
                t.buckets[nxt].key = key;
                __threadfence();
                atomicExch(&bk->next, nxt);
            } else {
                nxt = prev;
            }
        }
        for (int spin = 0; nxt == TG_LOCKED && spin < TG_MAX_SPIN; ++spin) {
            __nanosleep(64);
            nxt = *reinterpret_cast<volatile uint32_t*>(&bk->next);
        }
        if (nxt == TG_LOCKED) { atomicCAS(t.status, 0, (int)ADED_ERR_TIMEOUT); return; }
        if (nxt == 0) return;   // the allocating thread ran out of buckets and has reported it
        cur = nxt;
    }
    atomicCAS(t.status, 0, (int)ADED_ERR_TIMEOUT);
}

// Algorithm 2, one thread per window.  Duplicate windows inside one call are independent atomic
// adds, so the result is min(count + multiplicity, cap) whatever the thread order.
// `n_dev` (may be NULL): the span length lives on the device (at most n).
__global__ void k_tg_update(TgView t, const int32_t* __restrict__ tok, int n, const int32_t* __restrict__ n_dev) {
    const int i = blockIdx.x * blockDim.x + threadIdx.x + 2;
    if (n_dev && *n_dev < n) n = *n_dev;
    if (i >= n || *t.status != 0) return;
    const int a = tok[i - 2], b = tok[i - 1], c = tok[i];
    if (a < 0 || b < 0 || c < 0 || a >= t.vocab || b >= t.vocab || c >= t.vocab) {
        atomicCAS(t.status, 0, (int)ADED_ERR_INVALID_ARG);
        return;
    }
    tg_add(t, a, b, c, 1u);
}

// Every stored tri-gram with count >= min_count as (a, b, c) and its count, in no particular order;
// *n_out counts all of them, only the first `max_entries` are written.
__global__ void k_tg_export(TgView t, uint32_t min_count, int32_t* __restrict__ keys, uint32_t* __restrict__ counts,
                            unsigned long long max_entries, unsigned long long* n_out) {
    const size_t n = (size_t)t.n_home + t.n_over;
    for (size_t i = blockIdx.x * (size_t)blockDim.x + threadIdx.x; i < n; i += (size_t)gridDim.x * blockDim.x) {
        const Bucket* bk = t.buckets + i;
        const unsigned long long key = bk->key;
        if (key == TG_EMPTY) continue;
        for (int e = 0; e < 6; ++e) {
            const int32_t tk = bk->e[e].tok;
            const uint32_t cn = bk->e[e].cnt;
            if (tk < 0 || cn < min_count || cn == 0) continue;
            const unsigned long long at = atomicAdd(n_out, 1ull);
            if (at < max_entries) {
                keys[3 * at + 0] = (int32_t)(key >> 32);
                keys[3 * at + 1] = (int32_t)(key & 0xFFFFFFFFu);
                keys[3 * at + 2] = tk;
                counts[at] = cn;
            }
        }
    }
}

// Adds exported entries to a table (counts add up, saturating).
__global__ void k_tg_import(TgView t, const int32_t* __restrict__ keys, const uint32_t* __restrict__ counts, unsigned long long n) {
    const unsigned long long i = blockIdx.x * (unsigned long long)blockDim.x + threadIdx.x;
    if (i >= n || *t.status != 0) return;
    const int a = keys[3 * i], b = keys[3 * i + 1], c = keys[3 * i + 2];
    uint32_t inc = counts[i];
    if (a < 0 || b < 0 || c < 0 || a >= t.vocab || b >= t.vocab || c >= t.vocab) {
        atomicCAS(t.status, 0, (int)ADED_ERR_INVALID_ARG);
        return;
    }
    if (inc == 0) return;
    if (inc > t.cap) inc = t.cap;
    tg_add(t, a, b, c, inc);
}

// One selection round of a warp over the chain that starts at `home`: the largest packed
// (count, ~token) strictly below `prev`, or 0 when nothing is left; `total` = sum of the counts.
__device__ __forceinline__ unsigned long long tg_select_round(const TgView& t, int64_t home, unsigned long long prev,
                                                              int lane, uint32_t* total_out) {
    unsigned long long best = 0;
    uint32_t total = 0;
    int64_t cur = home;
    for (uint32_t hop = 0; cur >= 0 && hop <= t.n_over; ++hop) {
        const Bucket* bk = t.buckets + cur;
        if (lane < 6) {
            const int32_t tk = bk->e[lane].tok;
            const uint32_t cn = bk->e[lane].cnt;
            if (tk >= 0) {
                total += cn;
                const unsigned long long key = ((unsigned long long)cn << 32) | (0xFFFFFFFFu - (uint32_t)tk);
                if (cn >= t.min_count && cn > 0 && key < prev && key > best) best = key;
            }
        }
        const uint32_t nxt = bk->next;
        cur = nxt == 0 ? -1 : (int64_t)nxt;
    }
    for (int o = 16; o > 0; o >>= 1) {
        const unsigned long long ob = __shfl_xor_sync(0xffffffffu, best, o);
        if (ob > best) best = ob;
        total += __shfl_xor_sync(0xffffffffu, total, o);
    }
    if (total_out) *total_out = total;
    return best;
}

// The k <= TG_LIST largest packed (count, ~token) keys of the chain that starts at `home`, in descending order
// (count descending, token ascending among equals), in ONE walk over the chain: lanes 0..5 each keep the best
// TG_LIST keys of their entry slot of every bucket in registers (sorted insertion); afterwards the six lists
// are merged by k warp-wide maxima, the lane that held a maximum dropping it.  Keys are distinct (a context
// holds a token once).  Every lane returns the same list in `out` (0 = nothing left); `total` = sum of the counts.
constexpr int TG_LIST = 8;
static_assert(TG_LIST >= ADED_DRAFT_MAX_K, "the draft tree takes its lists in one walk");
__device__ __forceinline__ void tg_select_list(const TgView& t, int64_t home, int k, int lane,
                                               unsigned long long (&out)[TG_LIST], uint32_t* total_out) {
    unsigned long long loc[TG_LIST];
#pragma unroll
    for (int i = 0; i < TG_LIST; ++i) loc[i] = 0;
    uint32_t total = 0;
    int64_t cur = home;
    for (uint32_t hop = 0; cur >= 0 && hop <= t.n_over; ++hop) {
        const Bucket* bk = t.buckets + cur;
        if (lane < 6) {
            const int32_t tk = bk->e[lane].tok;
            const uint32_t cn = bk->e[lane].cnt;
            if (tk >= 0) {
                total += cn;
                unsigned long long key = ((unsigned long long)cn << 32) | (0xFFFFFFFFu - (uint32_t)tk);
                if (cn >= t.min_count && cn > 0 && key > loc[TG_LIST - 1]) {
#pragma unroll
                    for (int i = 0; i < TG_LIST; ++i) {       // sorted insertion: the key sinks to its place
                        if (key > loc[i]) { const unsigned long long tmp = loc[i]; loc[i] = key; key = tmp; }
                    }
                }
            }
        }
        const uint32_t nxt = bk->next;
        cur = nxt == 0 ? -1 : (int64_t)nxt;
    }
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) total += __shfl_xor_sync(0xffffffffu, total, o);
    if (total_out) *total_out = total;
#pragma unroll
    for (int r = 0; r < TG_LIST; ++r) {
        unsigned long long best = 0;
        if (r < k) {
            best = loc[0];
#pragma unroll
            for (int o = 16; o > 0; o >>= 1) {
                const unsigned long long ob = __shfl_xor_sync(0xffffffffu, best, o);
                if (ob > best) best = ob;
            }
            if (best != 0 && loc[0] == best) {                // this lane held it: drop it
#pragma unroll
                for (int i = 0; i + 1 < TG_LIST; ++i) loc[i] = loc[i + 1];
                loc[TG_LIST - 1] = 0;
            }
        }
        out[r] = best;
    }
}

// One warp per query.  Up to TG_LIST continuations: one walk over the context's chain (tg_select_list).  Longer
// lists: k selection rounds, a round picking the largest packed (count, ~token) strictly below the previous
// pick, which yields count descending, token ascending among equals, without storing the list.
__global__ void k_tg_topk(TgView t, const int32_t* __restrict__ ctx, int q, int k, int32_t* __restrict__ out_tok,
                          uint32_t* __restrict__ out_cnt, uint32_t* __restrict__ out_total) {
    const int w = (blockIdx.x * blockDim.x + threadIdx.x) >> 5;
    const int lane = threadIdx.x & 31;
    if (w >= q) return;
    const int a = ctx[2 * w], b = ctx[2 * w + 1];
    int64_t home = -1;
    if (a >= 0 && b >= 0 && a < t.vocab && b < t.vocab) home = tg_find_home(t, tg_key(a, b), false);
    if (k <= TG_LIST) {
        unsigned long long list[TG_LIST];
        uint32_t total;
        tg_select_list(t, home, k, lane, list, &total);
        if (lane == 0) {
#pragma unroll
            for (int r = 0; r < TG_LIST; ++r) {
                if (r < k) {
                    out_tok[(size_t)w * k + r] = list[r] ? (int32_t)(0xFFFFFFFFu - (uint32_t)list[r]) : -1;
                    out_cnt[(size_t)w * k + r] = (uint32_t)(list[r] >> 32);
                }
            }
            if (out_total) out_total[w] = total;
        }
        return;
    }
    unsigned long long prev = ~0ull;
    for (int round = 0; round < k; ++round) {
        uint32_t total;
        const unsigned long long best = tg_select_round(t, home, prev, lane, &total);
        if (lane == 0) {
            out_tok[(size_t)w * k + round] = best ? (int32_t)(0xFFFFFFFFu - (uint32_t)best) : -1;
            out_cnt[(size_t)w * k + round] = (uint32_t)(best >> 32);
            if (round == 0 && out_total) out_total[w] = total;
        }
        prev = best ? best : 0;   // nothing left: later rounds find nothing either
    }
}

// Draft tree of n_nodes nodes for the context (ctx[0], ctx[1]); one block of 32 warps.
// Level by level: every node of the current level gets its top-k list (one warp per node), then
// one thread appends the lists in node order, rank order -- the same tree as visiting the nodes in
// index order.  The filler pass (one thread; child lists kept in shared memory) hangs caller-
// supplied tokens under nodes with room, round-robin, until the tree is full.
constexpr int DRAFT_MAX_FILLER = 4 * ADED_MAX_NODES;

// Filler pass of one thread over a tree held in shared memory (tok, par, dep; kid[p][0 .. nkid[p]) the
// child tokens of node p): nodes are visited round-robin, a visited node with depth < max_depth and
// fewer than k children gets the next filler token none of its children holds.  Returns the new node
// count; *fail when the filler runs out, holds a token outside the vocabulary, or no node has room.
__device__ __forceinline__ int draft_fill(int32_t* tok, int32_t* par, int32_t* dep, int32_t* nkid, int32_t* kid, int n, int n_nodes,
                                          int max_depth, int k, const int32_t* fill, int n_filler, int vocab, bool* fail) {
    int pos = 0, p = 0, idle = 0;
    while (n < n_nodes) {
        const int nk = nkid[p];
        if (dep[p] < max_depth && nk < k) {
            int32_t f = -1;
            for (; pos < n_filler; ++pos) {
                f = fill[pos];
                bool clash = false;
                for (int j = 0; j < nk; ++j) clash |= kid[p * ADED_DRAFT_MAX_K + j] == f;
                if (!clash) break;
            }
            if (pos >= n_filler || f < 0 || f >= vocab) { *fail = true; break; }
            ++pos;
            kid[p * ADED_DRAFT_MAX_K + nk] = f;
            nkid[p] = nk + 1;
            tok[n] = f;
            par[n] = p;
            dep[n] = dep[p] + 1;
            nkid[n] = 0;
            ++n;
            idle = 0;
        } else if (++idle > n) {
            *fail = true;
            break;
        }
        p = (p + 1) % n;
    }
    return n;
}

__global__ void __launch_bounds__(1024)
k_draft_tree(TgView t, const int32_t* __restrict__ ctx, int n_nodes, int max_depth, int k,
             const int32_t* __restrict__ filler, int n_filler, int32_t* __restrict__ out_tok,
             int32_t* __restrict__ out_par, int32_t* __restrict__ out_real) {
    __shared__ int32_t s_tok[ADED_MAX_NODES], s_par[ADED_MAX_NODES], s_dep[ADED_MAX_NODES], s_nkid[ADED_MAX_NODES];
    __shared__ int32_t s_cand[ADED_MAX_NODES * ADED_DRAFT_MAX_K];   // top-k lists, later the child tokens of every node
    __shared__ int32_t s_fill[DRAFT_MAX_FILLER];
    __shared__ int s_n, s_lo, s_hi, s_fail;
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int prev_token = ctx[0];
    if (threadIdx.x == 0) {
        s_tok[0] = ctx[1];
        s_par[0] = -1;
        s_dep[0] = 0;
        s_n = 1;
        s_lo = 0;
        s_hi = 1;
        s_fail = 0;
    }
    for (int i = threadIdx.x; i < n_filler; i += blockDim.x) s_fill[i] = filler[i];
    for (int i = threadIdx.x; i < ADED_MAX_NODES; i += blockDim.x) s_nkid[i] = 0;
    __syncthreads();
    for (int d = 0; d < max_depth; ++d) {
        const int lo = s_lo, hi = s_hi;
        if (lo >= hi || s_n >= n_nodes) break;
        for (int node = lo + warp; node < hi; node += 32) {
            const int u = node == 0 ? prev_token : s_tok[s_par[node]], w = s_tok[node];
            int64_t home = -1;
            if (u >= 0 && w >= 0 && u < t.vocab && w < t.vocab) home = tg_find_home(t, tg_key(u, w), false);
            unsigned long long list[TG_LIST];          // (k <= ADED_DRAFT_MAX_K = TG_LIST: one walk over the chain)
            tg_select_list(t, home, k, lane, list, nullptr);
            if (lane == 0) {
#pragma unroll
                for (int r = 0; r < TG_LIST; ++r)
                    if (r < k) s_cand[node * ADED_DRAFT_MAX_K + r] = list[r] ? (int32_t)(0xFFFFFFFFu - (uint32_t)list[r]) : -1;
            }
        }
        __syncthreads();
        if (threadIdx.x == 0) {
            int n = s_n;
            for (int node = lo; node < hi && n < n_nodes; ++node) {
                for (int j = 0; j < k && n < n_nodes; ++j) {
                    const int32_t c = s_cand[node * ADED_DRAFT_MAX_K + j];
                    if (c < 0) break;
                    s_tok[n] = c;
                    s_par[n] = node;
                    s_dep[n] = d + 1;
                    s_nkid[node] = j + 1;    // s_cand[node][0 .. j] are this node's child tokens
                    ++n;
                }
            }
            s_lo = hi;
            s_hi = n;
            s_n = n;
        }
        __syncthreads();
    }
    if (threadIdx.x == 0) {
        int n = s_n;
        if (out_real) *out_real = n;
        if (filler && n < n_nodes) {
            bool fail = false;
            n = draft_fill(s_tok, s_par, s_dep, s_nkid, s_cand, n, n_nodes, max_depth, k, s_fill, n_filler, t.vocab, &fail);
            if (fail) s_fail = 1;
            s_n = n;
        }
        if (s_fail) atomicCAS(t.status, 0, (int)ADED_ERR_INVALID_ARG);
    }
    __syncthreads();
    const int n = s_n;
    for (int i = threadIdx.x; i < n_nodes; i += blockDim.x) {
        out_tok[i] = (i < n && !(s_fail && i == 0)) ? s_tok[i] : -1;
        out_par[i] = i < n ? s_par[i] : -1;
    }
}

// After a verification step: the span the table learns from (context + emitted tokens) and the
// context of the next step.  A failed step (accept length < 1) leaves the context and an empty span.
__global__ void k_decode_advance(const int32_t* __restrict__ out_tok, int32_t* __restrict__ out_len, int32_t* ctx,
                                 int32_t* __restrict__ span, int32_t* __restrict__ span_len, int max_emit) {
    __shared__ int32_t s_ctx[2];
    int a = *out_len;
    if (a > max_emit) a = max_emit;
    if (threadIdx.x < 2) s_ctx[threadIdx.x] = ctx[threadIdx.x];
    __syncthreads();
    if (a < 1) {
        if (threadIdx.x == 0) { *span_len = 0; *out_len = 0; }
        return;
    }
    for (int i = threadIdx.x; i < a + 2; i += blockDim.x) span[i] = i < 2 ? s_ctx[i] : out_tok[i - 2];
    if (threadIdx.x == 0) {
        *span_len = a + 2;
        ctx[0] = a >= 2 ? out_tok[a - 2] : s_ctx[1];
        ctx[1] = out_tok[a - 1];
    }
}

__global__ void k_tg_get(TgView t, int a, int b, int c, uint32_t* out) {
    *out = 0;
    if (a < 0 || b < 0 || c < 0 || a >= t.vocab || b >= t.vocab || c >= t.vocab) return;
    int64_t cur = tg_find_home(t, tg_key(a, b), false);
    for (uint32_t hop = 0; cur >= 0 && hop <= t.n_over; ++hop) {
        const Bucket* bk = t.buckets + cur;
        for (int e = 0; e < 6; ++e)
            if (bk->e[e].tok == c) { *out = bk->e[e].cnt; return; }
        cur = bk->next == 0 ? -1 : (int64_t)bk->next;
    }
}

__global__ void k_tg_stats(TgView t, unsigned long long* out) {
    unsigned long long entries = 0, used = 0;
    const size_t n = (size_t)t.n_home + t.n_over;
    for (size_t i = blockIdx.x * (size_t)blockDim.x + threadIdx.x; i < n; i += (size_t)gridDim.x * blockDim.x) {
        const Bucket* bk = t.buckets + i;
        int here = 0;
        for (int e = 0; e < 6; ++e) here += bk->e[e].tok >= 0;
        entries += here;
        used += bk->key != TG_EMPTY;
    }
    atomicAdd(out, entries);
    atomicAdd(out + 1, used);
}


// ---- draft maker: Monte Carlo tree search (Eq. 2-3, Algorithm 1) -----------------------------------
// One warp runs the search; every lane executes the same scalar logic on the tree in shared memory
// (lane 0 alone writes), the lanes cooperate only in the table lookups.  A lookup reads the context's
// chain once into shared memory and then selects the k best entries there.  Floating point is IEEE
// double, one rounded operation at a time (no fused multiply-add), so that the search can be
// reproduced bit for bit; the exploration factor E of Eq. 3 depends on an integer only and comes
// from a table the host computes.
constexpr int MC_MAX_ITER = 160, MC_MAX_K = ADED_DRAFT_MAX_K, MC_MAX_LEN = 8;
constexpr int MC_MAX_NODES = 1 + MC_MAX_ITER * MC_MAX_K;
constexpr int MC_CHAIN = 192;          // entries of a context held in shared memory (32 buckets)
constexpr int MC_CACHE = 64;           // remembered lookups (direct mapped): a search meets the same contexts again and again

struct McParams {
    int iterations, length, n_candidates, k;
    double e_table[MC_MAX_ITER + 1];   // E for sum N = 0 .. iterations
};

struct McLookup {                      // top-k list of one context
    int n;                             // valid entries
    int32_t word[MC_MAX_K];
    uint32_t count[MC_MAX_K];
    uint32_t total;                    // sum over ALL continuations of the context (Eq. 1's denominator)
};

// All 32 lanes call this with the same (a, b); the result is identical in every lane.
__device__ __forceinline__ void mc_lookup(const TgView& t, int a, int b, int k, int lane, int32_t* s_tok, uint32_t* s_cnt,
                                          McLookup& out) {
    out.n = 0;
    out.total = 0;
    int64_t home = -1;
    if (a >= 0 && b >= 0 && a < t.vocab && b < t.vocab) home = tg_find_home(t, tg_key(a, b), false);
    if (home < 0) return;
    // pass 1: the chain into shared memory (six entries per bucket, lanes 0..5 read them)
    int n_ent = 0;
    bool overflow = false;
    int64_t cur = home;
    for (uint32_t hop = 0; cur >= 0 && hop <= t.n_over; ++hop) {
        const Bucket* bk = t.buckets + cur;
        if (n_ent + 6 > MC_CHAIN) { overflow = true; break; }
        if (lane < 6) { s_tok[n_ent + lane] = bk->e[lane].tok; s_cnt[n_ent + lane] = bk->e[lane].cnt; }
        n_ent += 6;
        const uint32_t nxt = bk->next;
        cur = nxt == 0 ? -1 : (int64_t)nxt;
    }
    __syncwarp();
    unsigned long long prev = ~0ull;
    if (overflow) {                    // a very long chain: select round by round from global memory
        for (int round = 0; round < k; ++round) {
            uint32_t total;
            const unsigned long long best = tg_select_round(t, home, prev, lane, &total);
            out.total = total;
            if (!best) break;
            out.word[out.n] = (int32_t)(0xFFFFFFFFu - (uint32_t)best);
            out.count[out.n] = (uint32_t)(best >> 32);
            ++out.n;
            prev = best;
        }
        return;
    }
    uint32_t total = 0;
    for (int i = lane; i < n_ent; i += 32)
        if (s_tok[i] >= 0) total += s_cnt[i];
    for (int o = 16; o > 0; o >>= 1) total += __shfl_xor_sync(0xffffffffu, total, o);
    out.total = total;
    for (int round = 0; round < k; ++round) {
        unsigned long long best = 0;
        for (int i = lane; i < n_ent; i += 32) {
            const int32_t tk = s_tok[i];
            const uint32_t cn = s_cnt[i];
            if (tk < 0 || cn == 0 || cn < t.min_count) continue;
            const unsigned long long key = ((unsigned long long)cn << 32) | (0xFFFFFFFFu - (uint32_t)tk);
            if (key < prev && key > best) best = key;
        }
        for (int o = 16; o > 0; o >>= 1) {
            const unsigned long long ob = __shfl_xor_sync(0xffffffffu, best, o);
            if (ob > best) best = ob;
        }
        if (!best) break;
        out.word[out.n] = (int32_t)(0xFFFFFFFFu - (uint32_t)best);
        out.count[out.n] = (uint32_t)(best >> 32);
        ++out.n;
        prev = best;
    }
    __syncwarp();
}

// mc_lookup through the cache of remembered contexts (the table does not change during a search).
__device__ __forceinline__ void mc_lookup_cached(const TgView& t, int a, int b, int k, int lane, int32_t* s_tok, uint32_t* s_cnt,
                                                 unsigned long long* s_ckey, McLookup* s_cval, McLookup& out) {
    const unsigned long long key = tg_key(a, b);
    const int slot = (int)(tg_hash(key) & (MC_CACHE - 1));
    if (s_ckey[slot] == key) { out = s_cval[slot]; return; }
    mc_lookup(t, a, b, k, lane, s_tok, s_cnt, out);
    __syncwarp();
    if (lane == 0) { s_cval[slot] = out; s_ckey[slot] = key; }
    __syncwarp();
}

__host__ __device__ constexpr size_t mc_cache_offset() {
    return (((size_t)MC_MAX_NODES * (2 * 8 + 2 * 4 + 2 * 2 + 2 * 1) + (size_t)MC_CHAIN * 8 + ADED_MAX_NODES * 2) + 15) & ~(size_t)15;
}

__host__ __device__ constexpr size_t mc_fill_offset() {
    return (mc_cache_offset() + (size_t)MC_CACHE * (8 + sizeof(McLookup)) + (size_t)MC_MAX_ITER * MC_MAX_LEN * sizeof(float) + 15) & ~(size_t)15;
}

__global__ void __launch_bounds__(32)
k_mcts_draft(TgView t, const __grid_constant__ McParams p, const int32_t* __restrict__ ctx, const float* __restrict__ u,
             int32_t* __restrict__ out_tok, int32_t* __restrict__ out_par, int32_t* __restrict__ out_n,
             int32_t* __restrict__ sent_tok, double* __restrict__ sent_score, int32_t* __restrict__ out_n_sent,
             int n_target, const int32_t* __restrict__ filler, int n_filler) {
    extern __shared__ __align__(16) uint8_t mc_smem[];
    // 8-byte, then 4-byte, then 2-byte, then 1-byte arrays, so that each starts aligned
    double* s_score = reinterpret_cast<double*>(mc_smem);                 // [MC_MAX_NODES] sum of scores
    double* s_prior = s_score + MC_MAX_NODES;                             // Eq. 1 probability of the node's token in its parent's context
    int32_t* s_tok = reinterpret_cast<int32_t*>(s_prior + MC_MAX_NODES);  // token
    int32_t* s_visits = s_tok + MC_MAX_NODES;
    int32_t* s_ltok = s_visits + MC_MAX_NODES;                            // lookup scratch
    uint32_t* s_lcnt = reinterpret_cast<uint32_t*>(s_ltok + MC_CHAIN);
    int16_t* s_par = reinterpret_cast<int16_t*>(s_lcnt + MC_CHAIN);
    int16_t* s_first = s_par + MC_MAX_NODES;                              // first child (children are consecutive)
    int16_t* s_queue = s_first + MC_MAX_NODES;                            // [ADED_MAX_NODES] breadth-first order of the result
    uint8_t* s_nkid = reinterpret_cast<uint8_t*>(s_queue + ADED_MAX_NODES);
    uint8_t* s_flag = s_nkid + MC_MAX_NODES;                              // bit 0 expanded, bit 1 chosen, bit 2 kept
    unsigned long long* s_ckey = reinterpret_cast<unsigned long long*>(mc_smem + mc_cache_offset());   // [MC_CACHE] context of a remembered lookup
    McLookup* s_cval = reinterpret_cast<McLookup*>(s_ckey + MC_CACHE);
    for (int i = threadIdx.x; i < MC_CACHE; i += 32) s_ckey[i] = TG_EMPTY;
    float* s_u = reinterpret_cast<float*>(s_cval + MC_CACHE);            // the caller's uniform numbers
    for (int i = threadIdx.x; i < p.iterations * p.length; i += 32) s_u[i] = u[i];

    const int lane = threadIdx.x;
    const int prev_token = ctx[0], root_token = ctx[1];
    int n_nodes = 1;
    if (lane == 0) {
        s_tok[0] = root_token; s_par[0] = -1; s_first[0] = 0; s_nkid[0] = 0; s_flag[0] = 0;
        s_visits[0] = 0; s_score[0] = 0.0; s_prior[0] = 0.0;
    }
    __syncwarp();
    McLookup lk;
    for (int it = 0; it < p.iterations; ++it) {
        int node = 0, len = 1;
        int state[MC_MAX_LEN + 1];
        double sp[MC_MAX_LEN + 1];          // Eq. 1 probability of state[i] given its two predecessors
        state[0] = root_token;
        bool end = false;
        // selection
        while ((s_flag[node] & 1) && s_nkid[node] > 0 && !end) {
            // one lane per child (at most eight): the double divisions run side by side
            const int first = s_first[node], nk = s_nkid[node];
            const bool mine = lane < nk;
            const int c = first + (mine ? lane : 0);
            const int nv = mine ? s_visits[c] : 0;
            int n_sum = nv;
            for (int o = 16; o > 0; o >>= 1) n_sum += __shfl_xor_sync(0xffffffffu, n_sum, o);
            const double e = p.e_table[n_sum], root_n = sqrt((double)n_sum);
            const double q = nv ? __ddiv_rn(s_score[c], (double)nv) : 0.0;
            const double pr = s_prior[c];
            double best_s = __dadd_rn(q, __ddiv_rn(__dmul_rn(__dmul_rn(e, pr), root_n), __dadd_rn(1.0, (double)nv)));
            double best_p = pr;
            int best = mine ? c : -1;
            for (int o = 16; o > 0; o >>= 1) {
                const double os = __shfl_xor_sync(0xffffffffu, best_s, o), op = __shfl_xor_sync(0xffffffffu, best_p, o);
                const int ob = __shfl_xor_sync(0xffffffffu, best, o);
                if (ob >= 0 && (best < 0 || os > best_s || (os == best_s && ob < best))) { best = ob; best_s = os; best_p = op; }
            }
            node = best;
            state[len] = s_tok[node];
            sp[len] = best_p;
            ++len;
            if (len == p.length + 1) end = true;
        }
        // expansion
        if (!(s_flag[node] & 1) && !end) {
            const int a = node == 0 ? prev_token : s_tok[s_par[node]], b = s_tok[node];
            mc_lookup_cached(t, a, b, p.k, lane, s_ltok, s_lcnt, s_ckey, s_cval, lk);
            if (lane == 0) {
                s_flag[node] |= 1;
                s_first[node] = (int16_t)n_nodes;
                s_nkid[node] = (uint8_t)lk.n;
            }
            if (lane < lk.n) {                            // one lane per child: the divisions run side by side
                const int c = n_nodes + lane;
                s_tok[c] = lk.word[lane]; s_par[c] = (int16_t)node; s_first[c] = 0; s_nkid[c] = 0; s_flag[c] = 0;
                s_visits[c] = 0; s_score[c] = 0.0;
                s_prior[c] = __ddiv_rn((double)lk.count[lane], (double)lk.total);
            }
            __syncwarp();
            if (lk.n > 0) {
                n_nodes += lk.n;
                node = n_nodes - 1;                       // the last child created
                state[len] = s_tok[node];
                sp[len] = s_prior[node];
                ++len;
            }
        }
        // simulation
        int draws = 0;
        while (len < p.length + 1) {
            const int a = len >= 2 ? state[len - 2] : prev_token, b = state[len - 1];
            mc_lookup_cached(t, a, b, p.k, lane, s_ltok, s_lcnt, s_ckey, s_cval, lk);
            if (lk.n == 0) break;
            unsigned long long total = 0;
            for (int j = 0; j < lk.n; ++j) total += lk.count[j];
            unsigned long long u24 = __float2uint_rd(__fmul_rn(s_u[it * p.length + draws], 16777216.f));
            if (u24 > 16777215ull) u24 = 16777215ull;
            const unsigned long long target = (total * u24) >> 24;
            unsigned long long run = 0;
            int pick = lk.n - 1;
            for (int j = 0; j < lk.n; ++j) {
                run += lk.count[j];
                if (run > target) { pick = j; break; }
            }
            state[len] = lk.word[pick];
            sp[len] = __ddiv_rn((double)lk.count[pick], (double)lk.total);
            ++len;
            ++draws;
        }
        // back propagation
        double sc = 1.0;
        for (int i = 1; i < len; ++i) sc = __dadd_rn(sc, sp[i]);
        if (lane == 0) {
            for (int cur = node; cur >= 0; cur = s_par[cur]) {
                s_visits[cur] += 1;
                s_score[cur] = __dadd_rn(s_score[cur], sc);
            }
        }
        __syncwarp();
    }

    // ranking: leaves of the search tree by mean score (descending), earlier nodes first on ties
    int n_sent = 0;
    for (int r = 0; r < p.n_candidates; ++r) {
        double best_m = -1.0;
        int best_i = -1;
        for (int i = 1 + lane; i < n_nodes; i += 32) {
            if (s_nkid[i] != 0 || (s_flag[i] & 2)) continue;
            const double m = s_visits[i] ? __ddiv_rn(s_score[i], (double)s_visits[i]) : 0.0;
            if (best_i < 0 || m > best_m) { best_m = m; best_i = i; }     // i ascends within a lane: first wins ties
        }
        for (int o = 16; o > 0; o >>= 1) {
            const double om = __shfl_xor_sync(0xffffffffu, best_m, o);
            const int oi = __shfl_xor_sync(0xffffffffu, best_i, o);
            if (oi >= 0 && (best_i < 0 || om > best_m || (om == best_m && oi < best_i))) { best_m = om; best_i = oi; }
        }
        if (best_i < 0) break;
        if (lane == 0) {
            s_flag[best_i] |= 2;
            int path[MC_MAX_LEN], d = 0;
            for (int j = best_i; j > 0; j = s_par[j]) { s_flag[j] |= 4; path[d++] = s_tok[j]; }
            for (int j = 0; j < p.length; ++j) sent_tok[r * p.length + j] = j < d ? path[d - 1 - j] : -1;
            sent_score[r] = best_m;
        }
        __syncwarp();
        ++n_sent;
    }
    if (n_target > 0 && filler) {
        int32_t* f_fill = reinterpret_cast<int32_t*>(mc_smem + mc_fill_offset()) + ADED_MAX_NODES * (4 + ADED_DRAFT_MAX_K);
        for (int i = lane; i < n_filler; i += 32) f_fill[i] = filler[i];
        __syncwarp();
    }
    // prefix tree of the chosen sentences, breadth first, children in creation order
    if (lane == 0) {
        int count = 1;
        s_queue[0] = 0;
        out_tok[0] = root_token;
        out_par[0] = -1;
        for (int head = 0; head < count; ++head) {
            const int nd = s_queue[head];
            for (int c = s_first[nd]; c < s_first[nd] + s_nkid[nd]; ++c) {
                if (!(s_flag[c] & 4) || count >= ADED_MAX_NODES) continue;
                s_queue[count] = (int16_t)c;
                out_tok[count] = s_tok[c];
                out_par[count] = head;
                ++count;
            }
        }
        if (n_target > count && filler) {
            // complete the prefix tree to a fixed number of nodes, by the rule of the draft-tree kernel
            int32_t* f_tok = reinterpret_cast<int32_t*>(mc_smem + mc_fill_offset());       // [ADED_MAX_NODES] each
            int32_t* f_par = f_tok + ADED_MAX_NODES;
            int32_t* f_dep = f_par + ADED_MAX_NODES;
            int32_t* f_nkid = f_dep + ADED_MAX_NODES;
            int32_t* f_kid = f_nkid + ADED_MAX_NODES;                                      // [ADED_MAX_NODES][ADED_DRAFT_MAX_K]
            int32_t* f_fill = f_kid + ADED_MAX_NODES * ADED_DRAFT_MAX_K;                   // [DRAFT_MAX_FILLER], staged above by the whole warp
            for (int i = 0; i < count; ++i) { f_nkid[i] = 0; }
            for (int i = 0; i < count; ++i) {
                f_tok[i] = out_tok[i];
                f_par[i] = out_par[i];
                f_dep[i] = i == 0 ? 0 : f_dep[f_par[i]] + 1;
                if (i > 0) { const int pp = f_par[i]; f_kid[pp * ADED_DRAFT_MAX_K + f_nkid[pp]] = f_tok[i]; f_nkid[pp] += 1; }
            }
            bool fail = false;
            const int n2 = draft_fill(f_tok, f_par, f_dep, f_nkid, f_kid, count, n_target, p.length, p.k, f_fill, n_filler, t.vocab, &fail);
            for (int i = count; i < n2; ++i) { out_tok[i] = f_tok[i]; out_par[i] = f_par[i]; }
            count = n2;
            if (fail) { atomicCAS(t.status, 0, (int)ADED_ERR_INVALID_ARG); out_tok[0] = -1; }
        }
        *out_n = count;
        *out_n_sent = n_sent;
    }
}

static size_t mc_smem_bytes() {
    return mc_fill_offset() + (size_t)ADED_MAX_NODES * 4 * (4 + ADED_DRAFT_MAX_K) + (size_t)DRAFT_MAX_FILLER * 4 + 64;
}

}  // namespace aded

struct aded_trigram {
    aded_trigram_config cfg;
    int device;
    aded::TgView view;
    int32_t* stage_i;    // staging for the _host entry points
    uint32_t* stage_u;
    size_t stage_n;
    unsigned long long* stats_dev;
    int32_t* step_i;     // decoding step: span [ADED_MAX_NODES + 2], span length [1], filler staging
};

using namespace aded;

static constexpr size_t TG_STAGE = 1 << 16;
// step_i layout: span, span length, tokens from the table, filler staging
static constexpr int STEP_SPAN = 0, STEP_LEN = ADED_MAX_NODES + 2, STEP_REAL = STEP_LEN + 1, STEP_FILL = STEP_REAL + 1;
static constexpr int STEP_INTS = STEP_FILL + DRAFT_MAX_FILLER;

extern "C" {

aded_status aded_trigram_create(const aded_trigram_config* cfg, aded_trigram** out) {
    if (!cfg || !out) return ADED_ERR_INVALID_ARG;
    *out = nullptr;
    if (cfg->vocab < 1 || cfg->log2_buckets < 4 || cfg->log2_buckets > 28 || cfg->overflow_buckets < 0)
        return ADED_ERR_INVALID_ARG;
    if (cfg->cap > 0x7fffffffu) return ADED_ERR_INVALID_ARG;     // counts are kept below 2^31 so that concurrent adds cannot wrap
    aded_trigram* t = new (std::nothrow) aded_trigram();
    if (!t) return ADED_ERR_OOM;
    t->cfg = *cfg;
    t->stage_i = nullptr;
    t->stage_u = nullptr;
    t->stats_dev = nullptr;
    t->step_i = nullptr;
    t->view = TgView();
    const size_t n_home = (size_t)1 << cfg->log2_buckets, n = n_home + (size_t)cfg->overflow_buckets;
    bool ok = cudaGetDevice(&t->device) == cudaSuccess;
    cudaError_t e = cudaSuccess;
    if (ok) { e = cudaMalloc((void**)&t->view.buckets, n * sizeof(Bucket)); ok = e == cudaSuccess; }
    if (ok) ok = cudaMalloc((void**)&t->view.over_used, sizeof(uint32_t)) == cudaSuccess;
    if (ok) ok = cudaMalloc((void**)&t->view.status, sizeof(int32_t)) == cudaSuccess;
    if (ok) ok = cudaMalloc((void**)&t->stage_i, TG_STAGE * sizeof(int32_t)) == cudaSuccess;
    if (ok) ok = cudaMalloc((void**)&t->stage_u, TG_STAGE * sizeof(uint32_t)) == cudaSuccess;
    if (ok) ok = cudaMalloc((void**)&t->stats_dev, 2 * sizeof(unsigned long long)) == cudaSuccess;
    if (ok) ok = cudaMalloc((void**)&t->step_i, STEP_INTS * sizeof(int32_t)) == cudaSuccess;
    if (!ok) {
        cudaGetLastError();
        aded_trigram_destroy(t);
        return e == cudaErrorMemoryAllocation ? ADED_ERR_OOM : ADED_ERR_CUDA;
    }
    t->view.n_home = (uint32_t)n_home;
    t->view.n_home_mask = (uint32_t)n_home - 1;
    t->view.n_over = (uint32_t)cfg->overflow_buckets;
    t->view.vocab = cfg->vocab;
    t->view.cap = cfg->cap == 0 ? 0x7fffffffu : cfg->cap;
    t->view.min_count = cfg->min_count;
    k_tg_init<<<1024, 256>>>(t->view.buckets, n);
    ok = cudaMemset(t->view.over_used, 0, sizeof(uint32_t)) == cudaSuccess &&
         cudaMemset(t->view.status, 0, sizeof(int32_t)) == cudaSuccess && cudaDeviceSynchronize() == cudaSuccess;
    if (!ok) {
        cudaGetLastError();
        aded_trigram_destroy(t);
        return ADED_ERR_CUDA;
    }
    *out = t;
    return ADED_OK;
}

aded_status aded_trigram_destroy(aded_trigram* t) {
    if (!t) return ADED_ERR_INVALID_ARG;
    if (t->view.buckets) cudaFree(t->view.buckets);
    if (t->view.over_used) cudaFree(t->view.over_used);
    if (t->view.status) cudaFree(t->view.status);
    if (t->stage_i) cudaFree(t->stage_i);
    if (t->stage_u) cudaFree(t->stage_u);
    if (t->stats_dev) cudaFree(t->stats_dev);
    if (t->step_i) cudaFree(t->step_i);
    delete t;
    return ADED_OK;
}

aded_status aded_trigram_update(aded_trigram* t, const int32_t* tokens_dev, int32_t n, void* stream) {
    if (!t || n < 0 || (n > 0 && !tokens_dev)) return ADED_ERR_INVALID_ARG;
    if (n < 3) return ADED_OK;
    const int windows = n - 2;
    note_launch();
    k_tg_update<<<(windows + 255) / 256, 256, 0, static_cast<cudaStream_t>(stream)>>>(t->view, tokens_dev, n, nullptr);
    ADED_CUDA_TRY(cudaGetLastError());
    return ADED_OK;
}

aded_status aded_trigram_update_host(aded_trigram* t, const int32_t* tokens_host, int32_t n, void* stream) {
    if (!t || n < 0 || (n > 0 && !tokens_host)) return ADED_ERR_INVALID_ARG;
    if (n < 3) return ADED_OK;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    // long spans go through the staging buffer in pieces that overlap by two tokens
    for (int64_t lo = 0; lo + 2 < n; lo += (int64_t)TG_STAGE - 2) {
        const int64_t m = n - lo < (int64_t)TG_STAGE ? n - lo : (int64_t)TG_STAGE;
        ADED_CUDA_TRY(cudaMemcpyAsync(t->stage_i, tokens_host + lo, m * sizeof(int32_t), cudaMemcpyHostToDevice, st));
        aded_status s = aded_trigram_update(t, t->stage_i, (int32_t)m, stream);
        if (s != ADED_OK) return s;
        ADED_CUDA_TRY(cudaStreamSynchronize(st));
    }
    return ADED_OK;
}

aded_status aded_trigram_topk(const aded_trigram* t, const int32_t* ctx_dev, int32_t q, int32_t k,
                              int32_t* out_tokens_dev, uint32_t* out_counts_dev, uint32_t* out_total_dev,
                              void* stream) {
    if (!t || q < 0 || k < 1 || k > 32) return ADED_ERR_INVALID_ARG;
    if (q == 0) return ADED_OK;
    if (!ctx_dev || !out_tokens_dev || !out_counts_dev) return ADED_ERR_INVALID_ARG;
    const int warps_per_block = 4;
    note_launch();
    k_tg_topk<<<(q + warps_per_block - 1) / warps_per_block, warps_per_block * 32, 0, static_cast<cudaStream_t>(stream)>>>(
        t->view, ctx_dev, q, k, out_tokens_dev, out_counts_dev, out_total_dev);
    ADED_CUDA_TRY(cudaGetLastError());
    return ADED_OK;
}

aded_status aded_trigram_topk_host(const aded_trigram* t, const int32_t* ctx_host, int32_t q, int32_t k,
                                   int32_t* out_tokens_host, uint32_t* out_counts_host, uint32_t* out_total_host,
                                   void* stream) {
    if (!t || q < 0 || k < 1 || k > 32) return ADED_ERR_INVALID_ARG;
    if (q == 0) return ADED_OK;
    if (!ctx_host || !out_tokens_host || !out_counts_host) return ADED_ERR_INVALID_ARG;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    // staging: [ctx 2*qq | tokens qq*k] in stage_i, [counts qq*k | totals qq] in stage_u
    const int per = (int)(TG_STAGE / (size_t)(k + 2));
    for (int lo = 0; lo < q; lo += per) {
        const int qq = q - lo < per ? q - lo : per;
        int32_t* ctx_d = t->stage_i;
        int32_t* tok_d = t->stage_i + 2 * qq;
        uint32_t* cnt_d = t->stage_u;
        uint32_t* tot_d = t->stage_u + (size_t)qq * k;
        ADED_CUDA_TRY(cudaMemcpyAsync(ctx_d, ctx_host + 2 * (size_t)lo, 2 * (size_t)qq * sizeof(int32_t), cudaMemcpyHostToDevice, st));
        aded_status s = aded_trigram_topk(t, ctx_d, qq, k, tok_d, cnt_d, tot_d, stream);
        if (s != ADED_OK) return s;
        ADED_CUDA_TRY(cudaMemcpyAsync(out_tokens_host + (size_t)lo * k, tok_d, (size_t)qq * k * sizeof(int32_t), cudaMemcpyDeviceToHost, st));
        ADED_CUDA_TRY(cudaMemcpyAsync(out_counts_host + (size_t)lo * k, cnt_d, (size_t)qq * k * sizeof(uint32_t), cudaMemcpyDeviceToHost, st));
        if (out_total_host)
            ADED_CUDA_TRY(cudaMemcpyAsync(out_total_host + lo, tot_d, (size_t)qq * sizeof(uint32_t), cudaMemcpyDeviceToHost, st));
        ADED_CUDA_TRY(cudaStreamSynchronize(st));
    }
    return ADED_OK;
}

aded_status aded_draft_tree(const aded_trigram* t, const int32_t* context_dev, int32_t n_nodes, int32_t max_depth,
                            int32_t k, const int32_t* filler_dev, int32_t n_filler, int32_t* tree_tokens_dev,
                            int32_t* tree_parents_dev, int32_t* n_from_table_dev, void* stream) {
    if (!t || !context_dev || !tree_tokens_dev || !tree_parents_dev) return ADED_ERR_INVALID_ARG;
    if (n_nodes < 1 || n_nodes > ADED_MAX_NODES || max_depth < 0 || k < 1 || k > ADED_DRAFT_MAX_K) return ADED_ERR_INVALID_ARG;
    if (n_filler < 0 || n_filler > DRAFT_MAX_FILLER || (n_filler > 0 && !filler_dev)) return ADED_ERR_INVALID_ARG;
    note_launch();
    k_draft_tree<<<1, 1024, 0, static_cast<cudaStream_t>(stream)>>>(t->view, context_dev, n_nodes, max_depth, k,
                                                                    n_filler > 0 ? filler_dev : nullptr, n_filler,
                                                                    tree_tokens_dev, tree_parents_dev, n_from_table_dev);
    ADED_CUDA_TRY(cudaGetLastError());
    return ADED_OK;
}

aded_status aded_mcts_draft(const aded_trigram* t, const int32_t* context_dev, int32_t iterations, int32_t length,
                            int32_t n_candidates, int32_t k, float c1, float c2, const float* u_dev, int32_t* tree_tokens_dev,
                            int32_t* tree_parents_dev, int32_t* n_nodes_dev, int32_t* sentence_tokens_dev,
                            double* sentence_scores_dev, int32_t* n_sentences_dev, int32_t n_nodes_target,
                            const int32_t* filler_dev, int32_t n_filler, void* stream) {
    if (!t || !context_dev || !u_dev || !tree_tokens_dev || !tree_parents_dev || !n_nodes_dev || !sentence_tokens_dev ||
        !sentence_scores_dev || !n_sentences_dev)
        return ADED_ERR_INVALID_ARG;
    if (n_nodes_target < 0 || n_nodes_target > ADED_MAX_NODES || n_filler < 0 || n_filler > DRAFT_MAX_FILLER ||
        (n_nodes_target > 0 && (!filler_dev || n_filler < 1)))
        return ADED_ERR_INVALID_ARG;
    if (iterations < 1 || iterations > MC_MAX_ITER || length < 1 || length > MC_MAX_LEN || k < 1 || k > MC_MAX_K ||
        n_candidates < 1 || n_candidates * length + 1 > ADED_MAX_NODES || !(c2 > 0.f))
        return ADED_ERR_INVALID_ARG;
    static bool prepared = false;
    if (!prepared) {
        ADED_CUDA_TRY(cudaFuncSetAttribute(k_mcts_draft, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)mc_smem_bytes()));
        prepared = true;
    }
    McParams p;
    p.iterations = iterations;
    p.length = length;
    p.n_candidates = n_candidates;
    p.k = k;
    for (int n = 0; n <= MC_MAX_ITER; ++n) p.e_table[n] = (double)c1 + std::log(((double)n + (double)c2 + 1.0) / (double)c2);   // Eq. 3
    note_launch();
    k_mcts_draft<<<1, 32, mc_smem_bytes(), static_cast<cudaStream_t>(stream)>>>(t->view, p, context_dev, u_dev, tree_tokens_dev,
                                                                               tree_parents_dev, n_nodes_dev, sentence_tokens_dev,
                                                                               sentence_scores_dev, n_sentences_dev, n_nodes_target,
                                                                               n_nodes_target > 0 ? filler_dev : nullptr, n_filler);
    ADED_CUDA_TRY(cudaGetLastError());
    return ADED_OK;
}

aded_status aded_decode_step(aded_model* m, aded_kv* kv, aded_trigram* t, int32_t* context_dev, int32_t n_nodes,
                             int32_t max_depth, int32_t k, const int32_t* filler_dev, int32_t n_filler,
                             int32_t* out_tokens_dev, int32_t* out_accept_len_dev, int32_t* n_from_table_dev,
                             void* stream) {
    if (!m || !kv || !t || !context_dev || !out_tokens_dev || !out_accept_len_dev) return ADED_ERR_INVALID_ARG;
    if (n_nodes < 1 || n_nodes > ADED_MAX_NODES || n_nodes > m->cfg.max_rows) return ADED_ERR_INVALID_ARG;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    aded_status s = aded_draft_tree(t, context_dev, n_nodes, max_depth, k, filler_dev, n_filler, m->tokens, m->parents,
                                    n_from_table_dev ? n_from_table_dev : t->step_i + STEP_REAL, stream);
    if (s != ADED_OK) return s;
    s = aded_verify(m, kv, m->tokens, m->parents, n_nodes, out_tokens_dev, out_accept_len_dev, stream);
    if (s != ADED_OK) return s;
    note_launch(2);
    k_decode_advance<<<1, 160, 0, st>>>(out_tokens_dev, out_accept_len_dev, context_dev, t->step_i + STEP_SPAN,
                                        t->step_i + STEP_LEN, n_nodes);
    k_tg_update<<<(ADED_MAX_NODES + 255) / 256, 256, 0, st>>>(t->view, t->step_i + STEP_SPAN, n_nodes + 2,
                                                              t->step_i + STEP_LEN);
    ADED_CUDA_TRY(cudaGetLastError());
    return ADED_OK;
}

aded_status aded_decode_step_mcts(aded_model* m, aded_kv* kv, aded_trigram* t, int32_t* context_dev, int32_t n_nodes,
                                  int32_t iterations, int32_t length, int32_t n_candidates, int32_t k, float c1, float c2,
                                  const float* u_dev, const int32_t* filler_dev, int32_t n_filler, int32_t* out_tokens_dev,
                                  int32_t* out_accept_len_dev, void* stream) {
    if (!m || !kv || !t || !context_dev || !out_tokens_dev || !out_accept_len_dev) return ADED_ERR_INVALID_ARG;
    if (n_nodes < 1 || n_nodes > ADED_MAX_NODES || n_nodes > m->cfg.max_rows) return ADED_ERR_INVALID_ARG;
    if (!m->step_mcts) {      // sentences and counts of the search, which a decoding step does not hand out
        void* p = nullptr;
        ADED_CUDA_TRY(cudaMalloc(&p, (size_t)ADED_MAX_NODES * (sizeof(int32_t) + sizeof(double)) + 64));
        m->step_mcts = p;
        m->owned.push_back(p);
    }
    double* scores = reinterpret_cast<double*>(m->step_mcts);
    int32_t* sent = reinterpret_cast<int32_t*>(scores + ADED_MAX_NODES);
    int32_t* counts = t->step_i + STEP_REAL;          // found nodes; the sentence count goes to the span-length word, rewritten below
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    aded_status s = aded_mcts_draft(t, context_dev, iterations, length, n_candidates, k, c1, c2, u_dev, m->tokens, m->parents, counts,
                                    sent, scores, t->step_i + STEP_LEN, n_nodes, filler_dev, n_filler, stream);
    if (s != ADED_OK) return s;
    s = aded_verify(m, kv, m->tokens, m->parents, n_nodes, out_tokens_dev, out_accept_len_dev, stream);
    if (s != ADED_OK) return s;
    note_launch(2);
    k_decode_advance<<<1, 160, 0, st>>>(out_tokens_dev, out_accept_len_dev, context_dev, t->step_i + STEP_SPAN,
                                        t->step_i + STEP_LEN, n_nodes);
    k_tg_update<<<(ADED_MAX_NODES + 255) / 256, 256, 0, st>>>(t->view, t->step_i + STEP_SPAN, n_nodes + 2,
                                                              t->step_i + STEP_LEN);
    ADED_CUDA_TRY(cudaGetLastError());
    return ADED_OK;
}

aded_status aded_decode_step_host(aded_model* m, aded_kv* kv, aded_trigram* t, int32_t* context_dev, int32_t n_nodes,
                                  int32_t max_depth, int32_t k, const int32_t* filler_host, int32_t n_filler,
                                  int32_t* out_tokens_host, int32_t* out_accept_len_host, void* stream) {
    if (!m || !t || !out_tokens_host || !out_accept_len_host) return ADED_ERR_INVALID_ARG;
    if (n_filler < 0 || n_filler > DRAFT_MAX_FILLER || (n_filler > 0 && !filler_host)) return ADED_ERR_INVALID_ARG;
    if (n_nodes < 1 || n_nodes > m->cfg.max_rows) return ADED_ERR_INVALID_ARG;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    if (n_filler > 0)
        ADED_CUDA_TRY(cudaMemcpyAsync(t->step_i + STEP_FILL, filler_host, (size_t)n_filler * sizeof(int32_t),
                                      cudaMemcpyHostToDevice, st));
    const aded_status s = aded_decode_step(m, kv, t, context_dev, n_nodes, max_depth, k, t->step_i + STEP_FILL, n_filler,
                                           m->out_tokens, m->out_len, nullptr, stream);
    if (s != ADED_OK) return s;
    ADED_CUDA_TRY(cudaMemcpyAsync(out_tokens_host, m->out_tokens, (size_t)n_nodes * sizeof(int32_t), cudaMemcpyDeviceToHost, st));
    ADED_CUDA_TRY(cudaMemcpyAsync(out_accept_len_host, m->out_len, sizeof(int32_t), cudaMemcpyDeviceToHost, st));
    ADED_CUDA_TRY(cudaStreamSynchronize(st));
    return ADED_OK;
}

// ---- persistence and pruning -----------------------------------------------------------------------
aded_status aded_trigram_export(const aded_trigram* t, uint32_t min_count, int32_t* keys_dev, uint32_t* counts_dev,
                                uint64_t max_entries, uint64_t* n_out_host, void* stream) {
    if (!t || !n_out_host || (max_entries > 0 && (!keys_dev || !counts_dev))) return ADED_ERR_INVALID_ARG;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    unsigned long long n = 0;
    ADED_CUDA_TRY(cudaMemsetAsync(t->stats_dev, 0, sizeof n, st));
    note_launch();
    k_tg_export<<<1024, 256, 0, st>>>(t->view, min_count, keys_dev, counts_dev, max_entries, t->stats_dev);
    ADED_CUDA_TRY(cudaMemcpyAsync(&n, t->stats_dev, sizeof n, cudaMemcpyDeviceToHost, st));
    ADED_CUDA_TRY(cudaStreamSynchronize(st));
    *n_out_host = n;
    return ADED_OK;
}

aded_status aded_trigram_import(aded_trigram* t, const int32_t* keys_dev, const uint32_t* counts_dev, uint64_t n, void* stream) {
    if (!t || (n > 0 && (!keys_dev || !counts_dev))) return ADED_ERR_INVALID_ARG;
    if (n == 0) return ADED_OK;
    note_launch();
    k_tg_import<<<(unsigned int)((n + 255) / 256), 256, 0, static_cast<cudaStream_t>(stream)>>>(t->view, keys_dev, counts_dev, n);
    ADED_CUDA_TRY(cudaGetLastError());
    return ADED_OK;
}

aded_status aded_trigram_clear(aded_trigram* t, void* stream) {
    if (!t) return ADED_ERR_INVALID_ARG;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    note_launch();
    k_tg_init<<<1024, 256, 0, st>>>(t->view.buckets, (size_t)t->view.n_home + t->view.n_over);
    ADED_CUDA_TRY(cudaMemsetAsync(t->view.over_used, 0, sizeof(uint32_t), st));
    ADED_CUDA_TRY(cudaGetLastError());
    return ADED_OK;
}

// Scratch copy of the entries with count >= min_count; the caller frees *keys / *counts.
static aded_status tg_snapshot(const aded_trigram* t, uint32_t min_count, int32_t** keys, uint32_t** counts, uint64_t* n, void* stream) {
    *keys = nullptr;
    *counts = nullptr;
    uint64_t total = 0;
    aded_status s = aded_trigram_export(t, min_count, nullptr, nullptr, 0, &total, stream);
    if (s != ADED_OK) return s;
    *n = total;
    if (total == 0) return ADED_OK;
    if (cudaMalloc((void**)keys, total * 3 * sizeof(int32_t)) != cudaSuccess || cudaMalloc((void**)counts, total * sizeof(uint32_t)) != cudaSuccess) {
        cudaGetLastError();
        if (*keys) cudaFree(*keys);
        *keys = nullptr;
        return ADED_ERR_OOM;
    }
    uint64_t again = 0;
    s = aded_trigram_export(t, min_count, *keys, *counts, total, &again, stream);
    if (s == ADED_OK && again != total) s = ADED_ERR_INVALID_ARG;     // the table changed between the two passes
    if (s != ADED_OK) { cudaFree(*keys); cudaFree(*counts); *keys = nullptr; *counts = nullptr; }
    return s;
}

aded_status aded_trigram_prune(aded_trigram* t, uint32_t min_count, void* stream) {
    if (!t) return ADED_ERR_INVALID_ARG;
    int32_t* keys;
    uint32_t* counts;
    uint64_t n;
    aded_status s = tg_snapshot(t, min_count, &keys, &counts, &n, stream);
    if (s != ADED_OK) return s;
    s = aded_trigram_clear(t, stream);
    if (s == ADED_OK) s = aded_trigram_import(t, keys, counts, n, stream);
    cudaStreamSynchronize(static_cast<cudaStream_t>(stream));
    if (keys) cudaFree(keys);
    if (counts) cudaFree(counts);
    return s;
}

static const char TG_MAGIC[8] = {'A', 'D', 'E', 'D', 'T', 'G', '0', '1'};

aded_status aded_trigram_save(const aded_trigram* t, const char* path, void* stream) {
    if (!t || !path) return ADED_ERR_INVALID_ARG;
    int32_t* keys;
    uint32_t* counts;
    uint64_t n;
    aded_status s = tg_snapshot(t, 0, &keys, &counts, &n, stream);
    if (s != ADED_OK) return s;
    std::vector<int32_t> hk(n * 3);
    std::vector<uint32_t> hc(n);
    bool ok = true;
    if (n) {
        ok = cudaMemcpy(hk.data(), keys, n * 3 * sizeof(int32_t), cudaMemcpyDeviceToHost) == cudaSuccess &&
             cudaMemcpy(hc.data(), counts, n * sizeof(uint32_t), cudaMemcpyDeviceToHost) == cudaSuccess;
        cudaFree(keys);
        cudaFree(counts);
    }
    if (!ok) { cudaGetLastError(); return ADED_ERR_CUDA; }
    FILE* f = fopen(path, "wb");
    if (!f) return ADED_ERR_INVALID_ARG;
    const int32_t vocab = t->cfg.vocab;
    ok = fwrite(TG_MAGIC, 1, 8, f) == 8 && fwrite(&vocab, sizeof vocab, 1, f) == 1 && fwrite(&n, sizeof n, 1, f) == 1 &&
         (n == 0 || (fwrite(hk.data(), sizeof(int32_t), n * 3, f) == n * 3 && fwrite(hc.data(), sizeof(uint32_t), n, f) == n));
    ok = (fclose(f) == 0) && ok;
    return ok ? ADED_OK : ADED_ERR_INVALID_ARG;
}

aded_status aded_trigram_load(aded_trigram* t, const char* path, void* stream) {
    if (!t || !path) return ADED_ERR_INVALID_ARG;
    FILE* f = fopen(path, "rb");
    if (!f) return ADED_ERR_INVALID_ARG;
    char magic[8];
    int32_t vocab = 0;
    uint64_t n = 0;
    bool ok = fread(magic, 1, 8, f) == 8 && memcmp(magic, TG_MAGIC, 8) == 0 && fread(&vocab, sizeof vocab, 1, f) == 1 &&
              fread(&n, sizeof n, 1, f) == 1 && vocab == t->cfg.vocab && n <= ((uint64_t)1 << 34);
    std::vector<int32_t> hk;
    std::vector<uint32_t> hc;
    if (ok && n) {
        hk.resize(n * 3);
        hc.resize(n);
        ok = fread(hk.data(), sizeof(int32_t), n * 3, f) == n * 3 && fread(hc.data(), sizeof(uint32_t), n, f) == n;
    }
    fclose(f);
    if (!ok) return ADED_ERR_INVALID_ARG;
    if (n == 0) return ADED_OK;
    int32_t* keys = nullptr;
    uint32_t* counts = nullptr;
    if (cudaMalloc((void**)&keys, n * 3 * sizeof(int32_t)) != cudaSuccess || cudaMalloc((void**)&counts, n * sizeof(uint32_t)) != cudaSuccess) {
        cudaGetLastError();
        if (keys) cudaFree(keys);
        return ADED_ERR_OOM;
    }
    aded_status s = ADED_OK;
    if (cudaMemcpy(keys, hk.data(), n * 3 * sizeof(int32_t), cudaMemcpyHostToDevice) != cudaSuccess ||
        cudaMemcpy(counts, hc.data(), n * sizeof(uint32_t), cudaMemcpyHostToDevice) != cudaSuccess) {
        cudaGetLastError();
        s = ADED_ERR_CUDA;
    }
    if (s == ADED_OK) s = aded_trigram_import(t, keys, counts, n, stream);
    cudaStreamSynchronize(static_cast<cudaStream_t>(stream));
    cudaFree(keys);
    cudaFree(counts);
    return s;
}

aded_status aded_trigram_get(const aded_trigram* t, int32_t a, int32_t b, int32_t c, uint32_t* out_count_host, void* stream) {
    if (!t || !out_count_host) return ADED_ERR_INVALID_ARG;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    k_tg_get<<<1, 1, 0, st>>>(t->view, a, b, c, t->stage_u);
    ADED_CUDA_TRY(cudaMemcpyAsync(out_count_host, t->stage_u, sizeof(uint32_t), cudaMemcpyDeviceToHost, st));
    ADED_CUDA_TRY(cudaStreamSynchronize(st));
    return ADED_OK;
}

aded_status aded_trigram_stats(const aded_trigram* t, uint64_t* out_entries_host, uint64_t* out_buckets_host, void* stream) {
    if (!t || !out_entries_host || !out_buckets_host) return ADED_ERR_INVALID_ARG;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    unsigned long long res[2] = {0, 0};
    ADED_CUDA_TRY(cudaMemsetAsync(t->stats_dev, 0, sizeof res, st));
    k_tg_stats<<<1024, 256, 0, st>>>(t->view, t->stats_dev);
    ADED_CUDA_TRY(cudaMemcpyAsync(res, t->stats_dev, sizeof res, cudaMemcpyDeviceToHost, st));
    ADED_CUDA_TRY(cudaStreamSynchronize(st));
    *out_entries_host = res[0];
    *out_buckets_host = res[1];
    return ADED_OK;
}

aded_status aded_trigram_poll_status(aded_trigram* t, aded_status* out_host, void* stream) {
    if (!t || !out_host) return ADED_ERR_INVALID_ARG;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    int32_t v = 0;
    ADED_CUDA_TRY(cudaMemcpyAsync(&v, t->view.status, sizeof v, cudaMemcpyDeviceToHost, st));
    ADED_CUDA_TRY(cudaStreamSynchronize(st));
    if (v != 0) {
        ADED_CUDA_TRY(cudaMemsetAsync(t->view.status, 0, sizeof v, st));
        ADED_CUDA_TRY(cudaStreamSynchronize(st));
    }
    *out_host = static_cast<aded_status>(v);
    return ADED_OK;
}

}  // extern "C"
