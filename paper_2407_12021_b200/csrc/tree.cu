// Draft-tree bookkeeping around the forward pass ("Draft Construction and Verification"):
// validation + depths + ancestor masks before it, draft approval and cache compaction after it.
#include "aded_internal.cuh"

namespace aded {

// One block per sequence, one thread per node.  Checks that node 0 is the only root and every
// other node points at an earlier node, that tokens are in the vocabulary and that the cache has
// room; then each thread climbs from its node to the root, collecting the ancestor bit set and
// the depth.  The climb is bounded by the node count (parents decrease strictly).
__global__ void k_tree_prologue(const CallPtrs* __restrict__ call,
                                const int32_t* __restrict__ row_off, const int32_t* __restrict__ len,
                                const int32_t* __restrict__ cap, int vocab, int chain_mode,
                                RowMeta rows, int32_t* status) {
    pdl_enter();
    if (first_thread_of_grid()) trace_mark(status, TK_OTHER);
    const int32_t* __restrict__ tokens = call->tokens;
    const int32_t* __restrict__ parents = call->parents;
    const int b = blockIdx.x;
    const int off = row_off[b];
    const int T = row_off[b + 1] - off;
    const int i = threadIdx.x;
    __shared__ int s_bad;
    if (i == 0) s_bad = 0;
    __syncthreads();
    if (*status != 0) return;   // an earlier error is still pending: do nothing
    int p = -1;
    if (i < T) {
        p = chain_mode ? i - 1 : parents[off + i];
        const int t = tokens[off + i];
        if (t < 0 || t >= vocab) atomicMax(&s_bad, (int)ADED_ERR_INVALID_ARG);
        if (i == 0 ? (p != -1) : (p < 0 || p >= i)) atomicMax(&s_bad, (int)ADED_ERR_BAD_TREE);
    }
    if (i == 0 && len[b] + T > cap[b]) atomicMax(&s_bad, (int)ADED_ERR_KV_CAPACITY);
    __syncthreads();
    if (s_bad != 0) {
        if (i == 0) atomicCAS(status, 0, s_bad);
        return;
    }
    if (i < T) {
        uint64_t lo = 0, hi = 0;
        int depth = 0, cur = i;
        for (int step = 0; step < T; ++step) {
            if (cur < 64) lo |= 1ull << cur; else hi |= 1ull << (cur - 64);
            const int up = chain_mode ? cur - 1 : parents[off + cur];
            if (up < 0) break;
            cur = up;
            ++depth;
        }
        const int r = off + i;
        rows.seq[r] = b;
        rows.local[r] = i;
        rows.depth[r] = depth;
        rows.pos[r] = len[b] + depth;
        rows.anc[2 * r] = lo;
        rows.anc[2 * r + 1] = hi;
    }
}

// Draft approval, one thread per sequence (a tree has at most 128 nodes).  A node is approved when
// its parent is approved and its token equals the model's greedy token at the parent; the deepest
// approved node (lowest index among equals) ends the accepted path.  Emits the greedy token of
// every path node: the approved drafts' successors, ending with the model's own next token.
__global__ void k_accept(const CallPtrs* __restrict__ call,
                         const int32_t* __restrict__ row_off, const int32_t* __restrict__ best,
                         const int32_t* __restrict__ depth, const int32_t* __restrict__ len,
                         int32_t* __restrict__ path, int32_t* __restrict__ new_len,
                         const int32_t* status, int batch) {
    pdl_enter();
    if (first_thread_of_grid()) trace_mark(status, TK_PICK);
    const int32_t* __restrict__ tokens = call->tokens;
    const int32_t* __restrict__ parents = call->parents;
    int32_t* __restrict__ out_tokens = call->out_tokens;
    int32_t* __restrict__ out_len = call->out_len;
    const int out_stride = call->out_stride;
    // one block per sequence: the tree's arrays are fetched by all threads at once, then one thread walks
    const int b = blockIdx.x;
    if (b >= batch) return;
    __shared__ int32_t s_par[ADED_MAX_NODES], s_tok[ADED_MAX_NODES], s_best[ADED_MAX_NODES], s_dep[ADED_MAX_NODES];
    const int pass_status = *status;
    const int off = row_off[b];
    const int T = min(row_off[b + 1] - off, (int)ADED_MAX_NODES);
    for (int i = threadIdx.x; i < T; i += blockDim.x) {
        s_par[i] = parents[off + i];
        s_tok[i] = tokens[off + i];
        s_best[i] = best[off + i];
        s_dep[i] = depth[off + i];
    }
    __syncthreads();
    if (threadIdx.x != 0) return;
    approval_walk(s_par, s_tok, s_best, s_dep, T, pass_status, len[b], out_tokens + (size_t)b * out_stride, out_len + b,
                  path + b * ADED_MAX_NODES, new_len + b);
}

// Compaction: the tree's K/V were written at slots L + node index; the accepted path p_0 = 0 <
// p_1 < ... moves to slots L + 0, L + 1, ...  Because p_j >= j and the p_j increase, the source of a
// later move is never the destination of an earlier one, and a thread that owns one element
// column and walks j upwards reads every slot before it overwrites it.
template <typename T>
__global__ void k_compact(char* const* __restrict__ base, const int32_t* __restrict__ cap,
                          const int32_t* __restrict__ len, const int32_t* __restrict__ new_len,
                          const int32_t* __restrict__ path, int hd, const int32_t* status) {
    pdl_enter();
    if (first_thread_of_grid()) trace_mark(status, TK_OTHER);
    if (*status != 0) return;
    const int b = blockIdx.y;
    const int n_acc = new_len[b] - len[b];
    if (n_acc <= 1) return;
    const size_t plane = (size_t)blockIdx.x;   // (layer * 2 + k|v) * H + head
    T* p = reinterpret_cast<T*>(base[b]) + (plane * cap[b] + len[b]) * hd;
    for (int e = threadIdx.x; e < hd; e += blockDim.x) {
        for (int j = 1; j < n_acc; ++j) {
            const int src = path[b * ADED_MAX_NODES + j];
            if (!ADED_IN_RANGE(src >= j && src < ADED_MAX_NODES && len[b] + src < cap[b], status)) continue;
            if (src != j) p[(size_t)j * hd + e] = p[(size_t)src * hd + e];
        }
    }
}

__global__ void k_commit(int32_t* len, const int32_t* __restrict__ new_len, const int32_t* __restrict__ row_off,
                         int chain_mode, const int32_t* status, int batch) {
    pdl_enter();
    if (first_thread_of_grid()) trace_mark(status, TK_STEP_END);
    const int b = blockIdx.x * blockDim.x + threadIdx.x;
    if (b >= batch || *status != 0) return;
    len[b] = chain_mode ? len[b] + (row_off[b + 1] - row_off[b]) : new_len[b];
}

void launch_tree_prologue(aded_model* m, aded_kv* kv, int batch, int chain_mode, cudaStream_t st) {
    launch_k(k_tree_prologue, batch, ADED_MAX_NODES, 0, st, m->call_dev, m->seqs.row_off, kv->len_dev, kv->cap_dev,
                                                      m->cfg.vocab, chain_mode, m->rows, m->status);
}

void launch_accept(aded_model* m, aded_kv* kv, int batch, cudaStream_t st) {
    launch_k(k_accept, batch, 128, 0, st, m->call_dev, m->seqs.row_off, m->best, m->rows.depth,
                                               kv->len_dev, m->seqs.path, m->seqs.new_len, m->status, batch);
}

void launch_compact_commit(aded_model* m, aded_kv* kv, int batch, int chain_mode, cudaStream_t st) {
    if (!chain_mode) {
        dim3 grid(m->cfg.n_layers * 2 * m->cfg.n_heads, batch);
        if (m->cfg.dtype == ADED_BF16)
            launch_k(k_compact<bf16>, grid, 128, 0, st, kv->base_dev, kv->cap_dev, kv->len_dev, m->seqs.new_len,
                                                  m->seqs.path, m->cfg.head_dim, m->status);
        else
            launch_k(k_compact<float>, grid, 128, 0, st, kv->base_dev, kv->cap_dev, kv->len_dev, m->seqs.new_len,
                                                   m->seqs.path, m->cfg.head_dim, m->status);
    }
    launch_k(k_commit, (batch + 31) / 32, 32, 0, st, kv->len_dev, m->seqs.new_len, m->seqs.row_off, chain_mode,
                                               m->status, batch);
}

}  // namespace aded
