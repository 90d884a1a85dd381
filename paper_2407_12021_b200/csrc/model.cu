// Host side of the verification step: handles, argument checks and the launch sequence of one
// forward pass over a draft tree (see include/aded.h for the contract of every entry point).
#include <atomic>
#include <cstdio>
#include <cstdlib>
#include <cstring>
#include <new>

#include "aded_internal.cuh"

namespace aded {

static thread_local char g_last_cuda_error[256];

void note_cuda_error(cudaError_t e, const char* what) {
    snprintf(g_last_cuda_error, sizeof g_last_cuda_error, "%s: %s", what, cudaGetErrorString(e));
    if (getenv("ADED_VERBOSE")) fprintf(stderr, "[aded] CUDA error: %s\n", g_last_cuda_error);
    cudaGetLastError();
}

static std::atomic<uint64_t> g_launches{0};
void note_launch(int n) { g_launches.fetch_add((uint64_t)n, std::memory_order_relaxed); }

// Brackets a group of launches with events while profiling is on; otherwise only counts them.
struct Span {
    aded_model* m;
    cudaStream_t st;
    ProfSpan rec;
    bool on;
    Span(aded_model* m_, int group, int launches, cudaStream_t st_) : m(m_), st(st_), on(m_->prof_on) {
        note_launch(launches);
        if (!on) return;
        rec.group = group;
        rec.launches = launches;
        for (cudaEvent_t* e : {&rec.a, &rec.b}) {
            if (!m->prof_pool.empty()) { *e = m->prof_pool.back(); m->prof_pool.pop_back(); }
            else if (cudaEventCreate(e) != cudaSuccess) { on = false; cudaGetLastError(); return; }
        }
        cudaEventRecord(rec.a, st);
    }
    ~Span() {
        if (!on) return;
        cudaEventRecord(rec.b, st);
        m->prof_spans.push_back(rec);
    }
};

template <typename T>
static aded_status dev_alloc(aded_model* m, T** p, size_t count) {
    void* v = nullptr;
    cudaError_t e = cudaMalloc(&v, count * sizeof(T) > 0 ? count * sizeof(T) : 1);
    if (e != cudaSuccess) {
        cudaGetLastError();
        return e == cudaErrorMemoryAllocation ? ADED_ERR_OOM : ADED_ERR_CUDA;
    }
    m->owned.push_back(v);
    *p = static_cast<T*>(v);
    return ADED_OK;
}

#define TRY(expr) do { aded_status _s = (expr); if (_s != ADED_OK) return _s; } while (0)

static aded_status alloc_model(aded_model* m) {
    const aded_model_config& c = m->cfg;
    const size_t R = ((size_t)c.max_rows + 15) / 16 * 16, d = c.d_model, F = c.d_ffn, V = c.vocab, B = c.max_batch;
    size_t wide = 3 * d;
    if (2 * F > wide) wide = 2 * F;
    char* p;
    TRY(dev_alloc(m, &p, R * d * m->elem)); m->h = p;
    TRY(dev_alloc(m, &p, R * d * m->elem)); m->x = p;
    TRY(dev_alloc(m, &p, R * d * m->elem)); m->q = p;
    TRY(dev_alloc(m, &p, R * d * m->elem)); m->attn = p;
    TRY(dev_alloc(m, &p, R * F * m->elem)); m->act = p;
    TRY(dev_alloc(m, &m->y32, R * wide));
    TRY(dev_alloc(m, &m->logits, R * V));
    TRY(dev_alloc(m, &m->rope_cos, R * (c.head_dim / 2)));
    TRY(dev_alloc(m, &m->rope_sin, R * (c.head_dim / 2)));
    TRY(dev_alloc(m, &m->best, R));
    TRY(dev_alloc(m, &m->tokens, R));
    TRY(dev_alloc(m, &m->parents, R));
    TRY(dev_alloc(m, &m->out_tokens, R));
    TRY(dev_alloc(m, &m->out_len, B));
    TRY(dev_alloc(m, &m->status, (size_t)STATUS_WORDS));
    TRY(dev_alloc(m, &m->rows.seq, R));
    TRY(dev_alloc(m, &m->rows.local, R));
    TRY(dev_alloc(m, &m->rows.depth, R));
    TRY(dev_alloc(m, &m->rows.pos, R));
    TRY(dev_alloc(m, &m->rows.anc, 2 * R));
    TRY(dev_alloc(m, &m->seqs.row_off, B + 1));
    TRY(dev_alloc(m, &m->seqs.path, B * ADED_MAX_NODES));
    TRY(dev_alloc(m, &m->seqs.new_len, B));
    TRY(dev_alloc(m, &m->call_dev, 1));
    TRY(dev_alloc(m, &m->norm_ssq, R * 32));
    TRY(dev_alloc(m, &m->norm_count, R));
    TRY(dev_alloc(m, &m->argmax_val, R * ARGMAX_CHUNKS));
    TRY(dev_alloc(m, &m->argmax_idx, R * ARGMAX_CHUNKS));
    ADED_CUDA_TRY(cudaMemset(m->norm_count, 0, R * sizeof(int32_t)));
    if (d > 32 * 256) return ADED_ERR_UNSUPPORTED;   // the norm kernel keeps at most 32 column chunks per row
    ADED_CUDA_TRY(cudaMemset(m->status, 0, STATUS_WORDS * sizeof(int32_t)));
    ADED_CUDA_TRY(cudaMemset(m->h, 0, R * d * m->elem));
    ADED_CUDA_TRY(cudaMemset(m->x, 0, R * d * m->elem));
    ADED_CUDA_TRY(cudaMemset(m->attn, 0, R * d * m->elem));
    ADED_CUDA_TRY(cudaMemset(m->act, 0, R * F * m->elem));

    m->att_mma = c.dtype == ADED_BF16 && attn_prepare();
    // head_dim 128: the tcgen05 kernel (aded_debug_attention_kernel selects the mma.sync kernel, for comparisons)
    m->att_tc_ok = m->att_mma && attn_tc_supported(c) && attn_tc_prepare() && ws_make_map(&m->att_q_map, m->q, R, d, 64);
    m->att_tc = m->att_tc_ok;

    // tensor-core GEMM path: bf16 models whose every matrix tiles into 128-row x 64-column blocks
    m->ws_ready = false;
    if (c.dtype == ADED_BF16 && ws_supported(3 * (int)d, (int)d) && ws_supported((int)d, (int)d) && ws_supported(2 * (int)F, (int)d) &&
        ws_supported((int)d, (int)F) && ws_supported((int)V, (int)d)) {
        const int L = c.n_layers;
        m->ws_maps.resize(4 * L + 7);
        bool ok = ws_prepare();
        for (int l = 0; l < L && ok; ++l) {
            const aded_layer_weights& w = m->layers[l];
            ok = ws_make_map(&m->ws_maps[4 * l + WS_MAP_QKV], w.wqkv, 3 * d, d, 128) &&
                 ws_make_map(&m->ws_maps[4 * l + WS_MAP_O], w.wo, d, d, 128) &&
                 ws_make_map(&m->ws_maps[4 * l + WS_MAP_GU], w.wgu, 2 * F, d, 128) &&
                 ws_make_map(&m->ws_maps[4 * l + WS_MAP_D], w.wd, d, F, 128);
        }
        ok = ok && ws_make_map(&m->ws_maps[4 * L], m->top.lm_head, V, d, 128) &&
             ws_make_map(&m->ws_maps[4 * L + 1], m->x, R, d, 16) && ws_make_map(&m->ws_maps[4 * L + 2], m->attn, R, d, 16) &&
             ws_make_map(&m->ws_maps[4 * L + 3], m->act, R, F, 16) &&
             ws_make_map(&m->ws_maps[4 * L + 4], m->x, R, d, 64) && ws_make_map(&m->ws_maps[4 * L + 5], m->attn, R, d, 64) &&
             ws_make_map(&m->ws_maps[4 * L + 6], m->act, R, F, 64);
        if (ok) {
            // Private re-tiled copies of the weight matrices (as many bytes again as the matrices): each GEMM CTA
            // then reads one contiguous run of HBM instead of 128 strided lines per tile.  One allocation; when
            // the device has no room for it the GEMMs read the caller's row-major matrices through tensor maps.
            m->ws_tiled.assign(4 * L + 1, nullptr);
            m->ws_use_tiled = false;
            auto matrix = [&](int i, const void** src, size_t* nn, size_t* kk) {
                const int l = i / 4, kind = i % 4;
                if (i == 4 * L) { *src = m->top.lm_head; *nn = V; *kk = d; return; }
                const aded_layer_weights& w = m->layers[l];
                *src = kind == WS_MAP_QKV ? w.wqkv : kind == WS_MAP_O ? w.wo : kind == WS_MAP_GU ? w.wgu : w.wd;
                *nn = kind == WS_MAP_QKV ? 3 * d : kind == WS_MAP_O ? d : kind == WS_MAP_GU ? 2 * F : d;
                *kk = kind == WS_MAP_D ? F : d;
            };
            size_t total = 0;
            for (int i = 0; i < 4 * L + 1; ++i) {
                const void* src; size_t nn, kk;
                matrix(i, &src, &nn, &kk);
                total += nn * kk * 2;
            }
            uint8_t* pool = nullptr;
            if (dev_alloc(m, &pool, total) == ADED_OK) {
                size_t at = 0;
                for (int i = 0; i < 4 * L + 1; ++i) {
                    const void* src; size_t nn, kk;
                    matrix(i, &src, &nn, &kk);
                    ADED_CUDA_TRY(ws_retile(src, pool + at, (int)nn, (int)kk, nullptr));
                    m->ws_tiled[i] = pool + at;
                    at += nn * kk * 2;
                }
                ADED_CUDA_TRY(cudaDeviceSynchronize());
                m->ws_use_tiled = true;
            }
            size_t widest = 3 * d;
            if (2 * F > widest) widest = 2 * F;
            if (V > widest) widest = V;
            TRY(dev_alloc(m, &m->ws_slots, ws_slot_floats(m->device, (int)widest, (int)R)));
            // which slots make up each 128-column tile of each projection's result
            const int shapes[5][2] = {{3 * (int)d, (int)d}, {(int)d, (int)d}, {2 * (int)F, (int)d}, {(int)d, (int)F}, {(int)V, (int)d}};
            for (int i = 0; i < 5; ++i) {
                // O, gate/up and down launch one CTA per SM: their tiles then have half as many contributors and the
                // kernel that gathers them (residual + norm, SwiGLU), which is next on the critical path, reads half as
                // much (measured: two norms 12.8 -> 9.2 us per layer, the O and down GEMMs themselves unchanged).  QKV
                // keeps two (with one, the rotary step gains 0.8 us and the attention behind it loses 1.6), and so
                // does the LM head (its tail: 52.7 -> 58.8 us with one).
                m->ws_one_per_sm[i] = i == WS_MAP_O || i == WS_MAP_GU || i == WS_MAP_D;
                const int nt = shapes[i][0] / 128, kb = shapes[i][1] / 64, g = ws_grid(m->device, shapes[i][0], shapes[i][1], m->ws_one_per_sm[i]);
                std::vector<TileRef> table(nt);
                for (int t = 0; t < nt; ++t) table[t] = gemm_tile_ref(nt, kb, g, t);
                TRY(dev_alloc(m, &m->ws_tiles[i], (size_t)nt));
                ADED_CUDA_TRY(cudaMemcpy(m->ws_tiles[i], table.data(), nt * sizeof(TileRef), cudaMemcpyHostToDevice));
            }
            // the LM head's tail: one arrival counter per tile, per-tile greedy candidates of every row
            TRY(dev_alloc(m, &m->ws_counters, V / 128));
            ADED_CUDA_TRY(cudaMemset(m->ws_counters, 0, (V / 128) * sizeof(uint32_t)));
            m->ws_epoch = 0;
            TRY(dev_alloc(m, &m->cand_val, R * (V / 128)));
            TRY(dev_alloc(m, &m->cand_idx, R * (V / 128)));
            m->ws_ready = true;
        }
    }
    return ADED_OK;
}

// The launch sequence of one pass over `rows` rows.  chain_mode: the rows form a chain per sequence,
// every row is accepted and no logits are needed (prefill).
static aded_status enqueue_pass(aded_model* m, aded_kv* kv, const int32_t* offsets_src, int batch, int rows,
                                int max_tree, int chain_mode, cudaStream_t st) {
    const aded_model_config& c = m->cfg;
    const int d = c.d_model, F = c.d_ffn;
    const int xm = 4 * c.n_layers + 1;   // TMA descriptor indices of x, attn, act
    const bool ws = m->ws_ready;
    ADED_CUDA_TRY(cudaMemcpyAsync(m->seqs.row_off, offsets_src, (batch + 1) * sizeof(int32_t),
                                  cudaMemcpyHostToDevice, st));
    {
        const bool one = embed_norm_ws_supported(m);
        Span sp(m, PROF_OTHER, one ? 3 : 4, st);
        launch_tree_prologue(m, kv, batch, chain_mode, st);
        launch_rope_table(m, rows, st);
        if (one) {
            launch_embed_norm_ws(m, m->layers[0].norm1, rows, st);
        } else {
            launch_embed(m, rows, st);
            launch_add_rmsnorm(m, (const GemmOut*)nullptr, m->layers[0].norm1, rows, st);
        }
    }
    const size_t hid_bytes = (size_t)rows * d * m->elem;
    if (m->dbg_hidden) ADED_CUDA_TRY(cudaMemcpyAsync(m->dbg_hidden, m->h, hid_bytes, cudaMemcpyDeviceToDevice, st));
    const int passes = !ws ? 1 : rows > 128 ? (rows + 255) / 256 : 1;      // the tensor-core GEMM runs once per 128 rows (256 in calls with more)
    for (int l = 0; l < c.n_layers; ++l) {
        const aded_layer_weights& w = m->layers[l];
        const void* next_gain = l + 1 < c.n_layers ? m->layers[l + 1].norm1 : m->top.final_norm;
        auto wmap = [&](int which) { return ws ? 4 * l + which : -1; };      // TMA descriptor of a weight matrix (plain GEMM: none)
        GemmOut o;
        { Span sp(m, PROF_GEMM, passes, st); o = launch_gemm(m, wmap(WS_MAP_QKV), ws ? xm : -1, m->x, w.wqkv, m->y32, rows, 3 * d, d, WS_EPI_SLOTS, TK_GEMM_QKV, st); }
        { Span sp(m, PROF_OTHER, 1, st); launch_rope_kv(m, kv, o, l, rows, st); }
        { Span sp(m, PROF_ATTN, 1, st); launch_tree_attention(m, kv, l, batch, rows, max_tree, st); }
        { Span sp(m, PROF_GEMM, passes, st); o = launch_gemm(m, wmap(WS_MAP_O), ws ? xm + 1 : -1, m->attn, w.wo, m->y32, rows, d, d, WS_EPI_SLOTS, TK_GEMM_O, st); }
        { Span sp(m, PROF_OTHER, 1, st); launch_add_rmsnorm(m, &o, w.norm2, rows, st); }
        { Span sp(m, PROF_GEMM, passes, st); o = launch_gemm(m, wmap(WS_MAP_GU), ws ? xm : -1, m->x, w.wgu, m->y32, rows, 2 * F, d, WS_EPI_SLOTS, TK_GEMM_GU, st); }
        { Span sp(m, PROF_OTHER, 1, st); launch_swiglu(m, o, rows, st); }
        { Span sp(m, PROF_GEMM, passes, st); o = launch_gemm(m, wmap(WS_MAP_D), ws ? xm + 2 : -1, m->act, w.wd, m->y32, rows, d, F, WS_EPI_SLOTS, TK_GEMM_DOWN, st); }
        { Span sp(m, PROF_OTHER, 1, st); launch_add_rmsnorm(m, &o, next_gain, rows, st); }
        if (m->dbg_hidden)
            ADED_CUDA_TRY(cudaMemcpyAsync((char*)m->dbg_hidden + (size_t)(l + 1) * hid_bytes, m->h, hid_bytes,
                                          cudaMemcpyDeviceToDevice, st));
    }
    if (!chain_mode) {
        // The per-node logits are needed as a matrix only by the sampling mode and by a debug capture; the
        // greedy choice works from per-tile candidates left by the LM head's tail.
        const bool dense_logits = !ws || m->samp_on || m->dbg_logits;
        GemmOut lg;
        { Span sp(m, PROF_GEMM, passes, st);
          lg = launch_gemm(m, ws ? 4 * c.n_layers : -1, ws ? xm : -1, m->x, m->top.lm_head, m->logits, rows, c.vocab, d,
                           dense_logits ? WS_EPI_SLOTS : WS_EPI_ARGMAX, TK_GEMM_HEAD, st); }
        if (!dense_logits) {
            Span sp(m, PROF_OTHER, 1, st);
            launch_pick_accept(m, kv, batch, c.vocab / 128, st);
            if (m->dbg_best)
                ADED_CUDA_TRY(cudaMemcpyAsync(m->dbg_best, m->best, (size_t)rows * sizeof(int32_t), cudaMemcpyDeviceToDevice, st));
        } else {
            Span sp(m, PROF_OTHER, 3, st);
            if (m->samp_on) {
                // sampling mode: the logits as a dense matrix, then one drawn token per node in place of the greedy one
                launch_materialize(m, lg, m->logits, rows, st);
                ADED_CUDA_TRY(launch_sample_rows(m->logits, rows, c.vocab, c.vocab, m->samp_temp, m->samp_top_p, m->samp_u, m->best,
                                                 m->status, st));
            } else {
                launch_argmax(m, lg, rows, st);
            }
            if (m->dbg_logits) launch_materialize(m, lg, m->dbg_logits, rows, st);
            if (m->dbg_best)
                ADED_CUDA_TRY(cudaMemcpyAsync(m->dbg_best, m->best, (size_t)rows * sizeof(int32_t),
                                              cudaMemcpyDeviceToDevice, st));
            launch_accept(m, kv, batch, st);
        }
    }
    {
        Span sp(m, PROF_OTHER, chain_mode ? 1 : 2, st);
        launch_compact_commit(m, kv, batch, chain_mode, st);
    }
    ADED_CUDA_TRY(cudaGetLastError());
    return ADED_OK;
}

// One verify / append call: publish the caller's array pointers, then run the pass, kernel by kernel
// (every launch carries the programmatic-dependent-launch attribute).  Replaying a captured graph of the
// pass was measured slower for a caller that waits for each step (one graph launch of some 300 kernel
// nodes costs 2-4 ms of host time) and equal back to back, so there is no graph path.
static aded_status forward(aded_model* m, aded_kv* kv, const int32_t* tokens, const int32_t* parents,
                           const int32_t* offsets_host, int batch, int chain_mode, int32_t* out_tokens,
                           int out_stride, int32_t* out_len, cudaStream_t st) {
    const int rows = offsets_host[batch];
    int max_tree = 1;
    for (int b = 0; b < batch; ++b)
        if (offsets_host[b + 1] - offsets_host[b] > max_tree) max_tree = offsets_host[b + 1] - offsets_host[b];
    CallPtrs cp;
    cp.tokens = tokens;
    cp.parents = parents;
    cp.out_tokens = out_tokens;
    cp.out_len = out_len;
    cp.out_stride = out_stride;
    // pageable source: the runtime stages the bytes before returning, so the stack object may go
    ADED_CUDA_TRY(cudaMemcpyAsync(m->call_dev, &cp, sizeof cp, cudaMemcpyHostToDevice, st));
    const aded_status s = enqueue_pass(m, kv, offsets_host, batch, rows, max_tree, chain_mode, st);
    m->dbg_logits = nullptr;
    m->dbg_best = nullptr;
    m->dbg_hidden = nullptr;
    return s;
}

}  // namespace aded

using namespace aded;

extern "C" uint64_t aded_launch_count(void);

extern "C" {

aded_status aded_model_create(const aded_model_config* cfg, const aded_weights* weights, aded_model** out) {
    if (!cfg || !weights || !out || !weights->layers) return ADED_ERR_INVALID_ARG;
    *out = nullptr;
    if (cfg->n_layers < 1 || cfg->d_model < 1 || cfg->n_heads < 1 || cfg->d_ffn < 1 || cfg->vocab < 1 ||
        cfg->max_rows < 1 || cfg->max_batch < 1 || cfg->max_batch > cfg->max_rows)
        return ADED_ERR_INVALID_ARG;
    if (cfg->dtype != ADED_F32 && cfg->dtype != ADED_BF16) return ADED_ERR_INVALID_ARG;
    if (cfg->head_dim != 64 && cfg->head_dim != 128) return ADED_ERR_UNSUPPORTED;
    if (cfg->d_model != cfg->n_heads * cfg->head_dim) return ADED_ERR_INVALID_ARG;
    if (cfg->d_model % 16 || cfg->d_ffn % 16) return ADED_ERR_UNSUPPORTED;
    if (!weights->embed || !weights->final_norm || !weights->lm_head) return ADED_ERR_INVALID_ARG;
    for (int l = 0; l < cfg->n_layers; ++l) {
        const aded_layer_weights& w = weights->layers[l];
        if (!w.wqkv || !w.wo || !w.wgu || !w.wd || !w.norm1 || !w.norm2) return ADED_ERR_INVALID_ARG;
    }
    aded_model* m = new (std::nothrow) aded_model();
    if (!m) return ADED_ERR_OOM;
    m->cfg = *cfg;
    m->top = *weights;
    m->layers.assign(weights->layers, weights->layers + cfg->n_layers);
    m->top.layers = m->layers.data();
    m->elem = cfg->dtype == ADED_BF16 ? 2 : 4;
    m->dbg_logits = nullptr;
    m->dbg_best = nullptr;
    m->dbg_hidden = nullptr;
    m->step_mcts = nullptr;
    m->samp_on = false;
    m->samp_temp = 1.f;
    m->samp_top_p = 1.f;
    m->samp_u = nullptr;
    m->prof_on = false;
    m->call_dev = nullptr;
    m->ws_ready = false;
    m->ws_slots = nullptr;
    if (cudaGetDevice(&m->device) != cudaSuccess) {
        delete m;
        return ADED_ERR_CUDA;
    }
    aded_status s = alloc_model(m);
    if (s != ADED_OK) {
        aded_model_destroy(m);
        return s;
    }
    *out = m;
    return ADED_OK;
}

aded_status aded_model_destroy(aded_model* m) {
    if (!m) return ADED_ERR_INVALID_ARG;
    for (void* p : m->owned) cudaFree(p);
    for (ProfSpan& sp : m->prof_spans) { cudaEventDestroy(sp.a); cudaEventDestroy(sp.b); }
    for (cudaEvent_t e : m->prof_pool) cudaEventDestroy(e);
    delete m;
    return ADED_OK;
}

aded_status aded_kv_create(const aded_model* m, int32_t batch, const int32_t* capacity_host, aded_kv** out) {
    if (!m || !capacity_host || !out || batch < 1 || batch > m->cfg.max_batch) return ADED_ERR_INVALID_ARG;
    *out = nullptr;
    for (int b = 0; b < batch; ++b)
        if (capacity_host[b] < 1) return ADED_ERR_INVALID_ARG;
    aded_kv* kv = new (std::nothrow) aded_kv();
    if (!kv) return ADED_ERR_OOM;
    kv->model = m;
    kv->device = m->device;
    kv->batch = batch;
    kv->elem = m->elem;
    kv->cap.assign(capacity_host, capacity_host + batch);
    kv->base_dev = nullptr;
    kv->cap_dev = nullptr;
    kv->len_dev = nullptr;
    kv->maps_dev = nullptr;
    const aded_model_config& c = m->cfg;
    aded_status s = ADED_OK;
    for (int b = 0; b < batch && s == ADED_OK; ++b) {
        const size_t bytes = (size_t)c.n_layers * 2 * c.d_model * kv->cap[b] * kv->elem;
        void* p = nullptr;
        cudaError_t e = cudaMalloc(&p, bytes);
        if (e != cudaSuccess) {
            cudaGetLastError();
            s = e == cudaErrorMemoryAllocation ? ADED_ERR_OOM : ADED_ERR_CUDA;
            break;
        }
        kv->base.push_back(static_cast<char*>(p));
        // Zero-filled: rows past the last key are read (with probability exactly zero) by the attention
        // kernel's last key block and must hold finite values.
        if (cudaMemset(p, 0, bytes) != cudaSuccess) s = ADED_ERR_CUDA;
    }
    if (s == ADED_OK && m->att_tc_ok) {
        std::vector<CUtensorMap> maps(batch);
        for (int b = 0; b < batch && s == ADED_OK; ++b)
            if (!aded::attn_tc_make_kv_map(&maps[b], kv->base[b], (uint64_t)kv->cap[b], (uint64_t)c.n_layers * 2 * c.n_heads)) s = ADED_ERR_CUDA;
        if (s == ADED_OK && (cudaMalloc((void**)&kv->maps_dev, batch * sizeof(CUtensorMap)) != cudaSuccess ||
                             cudaMemcpy(kv->maps_dev, maps.data(), batch * sizeof(CUtensorMap), cudaMemcpyHostToDevice) != cudaSuccess))
            s = ADED_ERR_CUDA;
    }
    if (s == ADED_OK && (cudaMalloc((void**)&kv->base_dev, batch * sizeof(char*)) != cudaSuccess ||
                         cudaMalloc((void**)&kv->cap_dev, batch * sizeof(int32_t)) != cudaSuccess ||
                         cudaMalloc((void**)&kv->len_dev, batch * sizeof(int32_t)) != cudaSuccess))
        s = ADED_ERR_OOM;
    if (s == ADED_OK && (cudaMemcpy(kv->base_dev, kv->base.data(), batch * sizeof(char*), cudaMemcpyHostToDevice) != cudaSuccess ||
                         cudaMemcpy(kv->cap_dev, kv->cap.data(), batch * sizeof(int32_t), cudaMemcpyHostToDevice) != cudaSuccess ||
                         cudaMemset(kv->len_dev, 0, batch * sizeof(int32_t)) != cudaSuccess))
        s = ADED_ERR_CUDA;
    if (s != ADED_OK) {
        cudaGetLastError();
        aded_kv_destroy(kv);
        return s;
    }
    *out = kv;
    return ADED_OK;
}

aded_status aded_kv_destroy(aded_kv* kv) {
    if (!kv) return ADED_ERR_INVALID_ARG;
    for (char* p : kv->base) cudaFree(p);
    if (kv->base_dev) cudaFree(kv->base_dev);
    if (kv->cap_dev) cudaFree(kv->cap_dev);
    if (kv->len_dev) cudaFree(kv->len_dev);
    if (kv->maps_dev) cudaFree(kv->maps_dev);
    delete kv;
    return ADED_OK;
}

aded_status aded_kv_len(const aded_kv* kv, int32_t seq, int32_t* out_len_host, void* stream) {
    if (!kv || !out_len_host || seq < 0 || seq >= kv->batch) return ADED_ERR_INVALID_ARG;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    ADED_CUDA_TRY(cudaMemcpyAsync(out_len_host, kv->len_dev + seq, sizeof(int32_t), cudaMemcpyDeviceToHost, st));
    ADED_CUDA_TRY(cudaStreamSynchronize(st));
    return ADED_OK;
}

// Copies between the caller's [head][n_pos][hd] arrays and one layer's K and V planes.
static aded_status kv_copy(const aded_kv* kv, int seq, int layer, int pos0, int n_pos, void* k, void* v,
                           bool into_cache, cudaStream_t st) {
    const aded_model_config& c = kv->model->cfg;
    const size_t row = (size_t)c.head_dim * kv->elem;
    const size_t cap = kv->cap[seq];
    for (int which = 0; which < 2; ++which) {
        char* user = static_cast<char*>(which ? v : k);
        char* plane = kv->base[seq] + (((size_t)layer * 2 + which) * c.n_heads * cap + pos0) * row;
        // n_heads strided blocks of n_pos rows each
        if (into_cache)
            ADED_CUDA_TRY(cudaMemcpy2DAsync(plane, cap * row, user, (size_t)n_pos * row, (size_t)n_pos * row,
                                            c.n_heads, cudaMemcpyDeviceToDevice, st));
        else
            ADED_CUDA_TRY(cudaMemcpy2DAsync(user, (size_t)n_pos * row, plane, cap * row, (size_t)n_pos * row,
                                            c.n_heads, cudaMemcpyDeviceToDevice, st));
    }
    return ADED_OK;
}

aded_status aded_kv_load(aded_kv* kv, int32_t seq, int32_t layer, const void* k_dev, const void* v_dev,
                         int32_t n_pos, void* stream) {
    if (!kv || !k_dev || !v_dev || seq < 0 || seq >= kv->batch) return ADED_ERR_INVALID_ARG;
    if (layer < 0 || layer >= kv->model->cfg.n_layers || n_pos < 1) return ADED_ERR_INVALID_ARG;
    if (n_pos > kv->cap[seq]) return ADED_ERR_KV_CAPACITY;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    aded_status s = kv_copy(kv, seq, layer, 0, n_pos, const_cast<void*>(k_dev), const_cast<void*>(v_dev), true, st);
    if (s != ADED_OK) return s;
    ADED_CUDA_TRY(cudaMemcpyAsync(kv->len_dev + seq, &n_pos, sizeof(int32_t), cudaMemcpyHostToDevice, st));
    ADED_CUDA_TRY(cudaStreamSynchronize(st));   // n_pos is a stack variable
    return ADED_OK;
}

aded_status aded_kv_set_len(aded_kv* kv, int32_t seq, int32_t new_len, void* stream) {
    if (!kv || seq < 0 || seq >= kv->batch || new_len < 0) return ADED_ERR_INVALID_ARG;
    if (new_len > kv->cap[seq]) return ADED_ERR_KV_CAPACITY;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    ADED_CUDA_TRY(cudaMemcpyAsync(kv->len_dev + seq, &new_len, sizeof(int32_t), cudaMemcpyHostToDevice, st));
    ADED_CUDA_TRY(cudaStreamSynchronize(st));   // new_len is a stack variable
    return ADED_OK;
}

aded_status aded_kv_read(const aded_kv* kv, int32_t seq, int32_t layer, int32_t pos0, int32_t n_pos,
                         void* k_dev, void* v_dev, void* stream) {
    if (!kv || !k_dev || !v_dev || seq < 0 || seq >= kv->batch) return ADED_ERR_INVALID_ARG;
    if (layer < 0 || layer >= kv->model->cfg.n_layers || pos0 < 0 || n_pos < 1) return ADED_ERR_INVALID_ARG;
    if ((int64_t)pos0 + n_pos > kv->cap[seq]) return ADED_ERR_KV_CAPACITY;
    return kv_copy(kv, seq, layer, pos0, n_pos, k_dev, v_dev, false, static_cast<cudaStream_t>(stream));
}

aded_status aded_append(aded_model* m, aded_kv* kv, int32_t seq, const int32_t* tokens_dev, int32_t n, void* stream) {
    if (!m || !kv || !tokens_dev || kv->model != m) return ADED_ERR_INVALID_ARG;
    if (kv->batch != 1 || seq != 0) return ADED_ERR_UNSUPPORTED;
    if (n < 1 || n > ADED_MAX_NODES || n > m->cfg.max_rows) return ADED_ERR_INVALID_ARG;
    const int32_t off[2] = {0, n};
    return forward(m, kv, tokens_dev, nullptr, off, 1, 1, nullptr, 0, nullptr, static_cast<cudaStream_t>(stream));
}

aded_status aded_verify_batch(aded_model* m, aded_kv* kv, const int32_t* tree_offsets_host,
                              const int32_t* tree_tokens_dev, const int32_t* tree_parents_dev,
                              int32_t* out_tokens_dev, int32_t out_stride, int32_t* out_accept_len_dev,
                              void* stream) {
    if (!m || !kv || !tree_offsets_host || !tree_tokens_dev || !tree_parents_dev || !out_tokens_dev ||
        !out_accept_len_dev || kv->model != m)
        return ADED_ERR_INVALID_ARG;
    const int batch = kv->batch;
    if (tree_offsets_host[0] != 0) return ADED_ERR_INVALID_ARG;
    for (int b = 0; b < batch; ++b) {
        const int t = tree_offsets_host[b + 1] - tree_offsets_host[b];
        if (t < 1 || t > ADED_MAX_NODES || t > out_stride) return ADED_ERR_INVALID_ARG;
    }
    if (tree_offsets_host[batch] > m->cfg.max_rows) return ADED_ERR_INVALID_ARG;
    return forward(m, kv, tree_tokens_dev, tree_parents_dev, tree_offsets_host, batch, 0, out_tokens_dev,
                   out_stride, out_accept_len_dev, static_cast<cudaStream_t>(stream));
}

aded_status aded_verify(aded_model* m, aded_kv* kv, const int32_t* tree_tokens_dev,
                        const int32_t* tree_parents_dev, int32_t n_nodes, int32_t* out_tokens_dev,
                        int32_t* out_accept_len_dev, void* stream) {
    if (!kv || kv->batch != 1) return ADED_ERR_INVALID_ARG;
    if (n_nodes < 1 || n_nodes > ADED_MAX_NODES) return ADED_ERR_INVALID_ARG;
    const int32_t off[2] = {0, n_nodes};
    return aded_verify_batch(m, kv, off, tree_tokens_dev, tree_parents_dev, out_tokens_dev, n_nodes,
                             out_accept_len_dev, stream);
}

aded_status aded_verify_sampled(aded_model* m, aded_kv* kv, const int32_t* tree_tokens_dev,
                                const int32_t* tree_parents_dev, int32_t n_nodes, float temperature, float top_p,
                                const float* u_dev, int32_t* out_tokens_dev, int32_t* out_accept_len_dev, void* stream) {
    if (!m || !u_dev) return ADED_ERR_INVALID_ARG;
    if (!(temperature > 0.f) || !(top_p >= 1.f / 65536.f) || !(top_p <= 1.f)) return ADED_ERR_INVALID_ARG;
    if (!sample_supported(m->cfg.vocab)) return ADED_ERR_UNSUPPORTED;
    m->samp_on = true;
    m->samp_temp = temperature;
    m->samp_top_p = top_p;
    m->samp_u = u_dev;
    const aded_status s = aded_verify(m, kv, tree_tokens_dev, tree_parents_dev, n_nodes, out_tokens_dev, out_accept_len_dev, stream);
    m->samp_on = false;
    m->samp_u = nullptr;
    return s;
}

aded_status aded_verify_host(aded_model* m, aded_kv* kv, const int32_t* tree_tokens_host,
                             const int32_t* tree_parents_host, int32_t n_nodes, int32_t* out_tokens_host,
                             int32_t* out_accept_len_host, void* stream) {
    if (!m || !kv || !tree_tokens_host || !tree_parents_host || !out_tokens_host || !out_accept_len_host)
        return ADED_ERR_INVALID_ARG;
    if (n_nodes < 1 || n_nodes > ADED_MAX_NODES || n_nodes > m->cfg.max_rows) return ADED_ERR_INVALID_ARG;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    const size_t bytes = (size_t)n_nodes * sizeof(int32_t);
    ADED_CUDA_TRY(cudaMemcpyAsync(m->tokens, tree_tokens_host, bytes, cudaMemcpyHostToDevice, st));
    ADED_CUDA_TRY(cudaMemcpyAsync(m->parents, tree_parents_host, bytes, cudaMemcpyHostToDevice, st));
    aded_status s = aded_verify(m, kv, m->tokens, m->parents, n_nodes, m->out_tokens, m->out_len, stream);
    if (s != ADED_OK) return s;
    ADED_CUDA_TRY(cudaMemcpyAsync(out_tokens_host, m->out_tokens, bytes, cudaMemcpyDeviceToHost, st));
    ADED_CUDA_TRY(cudaMemcpyAsync(out_accept_len_host, m->out_len, sizeof(int32_t), cudaMemcpyDeviceToHost, st));
    ADED_CUDA_TRY(cudaStreamSynchronize(st));
    return ADED_OK;
}

aded_status aded_debug_gemm(aded_model* m, int32_t layer, int32_t which, const void* x_dev, int32_t rows,
                            float* y_dev, void* stream) {
    if (!m || !x_dev || !y_dev || which < 0 || which > 4 || rows < 1 || rows > m->cfg.max_rows)
        return ADED_ERR_INVALID_ARG;
    if (which < 4 && (layer < 0 || layer >= m->cfg.n_layers)) return ADED_ERR_INVALID_ARG;
    const aded_model_config& c = m->cfg;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    const int d = c.d_model, F = c.d_ffn, xm = 4 * c.n_layers + 1;
    const int n = which == 0 ? 3 * d : which == 2 ? 2 * F : which == 4 ? c.vocab : d;
    const int k = which == 3 ? F : d;
    void* xbuf = which == 1 ? m->attn : which == 3 ? m->act : m->x;
    const int x_map = which == 1 ? xm + 1 : which == 3 ? xm + 2 : xm;
    const void* w = which == 4 ? m->top.lm_head
                               : which == 0 ? m->layers[layer].wqkv
                                            : which == 1 ? m->layers[layer].wo
                                                         : which == 2 ? m->layers[layer].wgu : m->layers[layer].wd;
    const int w_map = which == 4 ? 4 * c.n_layers : 4 * layer + which;
    float* ybuf = which == 4 ? m->logits : m->y32;
    ADED_CUDA_TRY(cudaMemcpyAsync(xbuf, x_dev, (size_t)rows * k * m->elem, cudaMemcpyDeviceToDevice, st));
    note_launch();
    const GemmOut o = launch_gemm(m, m->ws_ready ? w_map : -1, m->ws_ready ? x_map : -1, xbuf, w, ybuf, rows, n, k, WS_EPI_SLOTS, TK_OTHER, st);
    launch_materialize(m, o, y_dev, rows, st);
    ADED_CUDA_TRY(cudaGetLastError());
    return ADED_OK;
}

aded_status aded_debug_capture_hidden(aded_model* m, void* hidden_dev) {
    if (!m) return ADED_ERR_INVALID_ARG;
    m->dbg_hidden = hidden_dev;
    return ADED_OK;
}

aded_status aded_debug_read_buffer(aded_model* m, int32_t which, int32_t rows, void* out_dev, void* stream) {
    if (!m || !out_dev || which < 0 || which > 4 || rows < 1 || rows > m->cfg.max_rows) return ADED_ERR_INVALID_ARG;
    const void* src = which == 0 ? m->h : which == 1 ? m->x : which == 2 ? m->q : which == 3 ? m->attn : m->act;
    const size_t width = which == 4 ? m->cfg.d_ffn : m->cfg.d_model;
    ADED_CUDA_TRY(cudaMemcpyAsync(out_dev, src, (size_t)rows * width * m->elem, cudaMemcpyDeviceToDevice,
                                  static_cast<cudaStream_t>(stream)));
    return ADED_OK;
}

aded_status aded_debug_capture(aded_model* m, float* logits_dev, int32_t* best_dev) {
    if (!m) return ADED_ERR_INVALID_ARG;
    m->dbg_logits = logits_dev;
    m->dbg_best = best_dev;
    return ADED_OK;
}

aded_status aded_profile_begin(aded_model* m) {
    if (!m) return ADED_ERR_INVALID_ARG;
    for (ProfSpan& sp : m->prof_spans) { m->prof_pool.push_back(sp.a); m->prof_pool.push_back(sp.b); }
    m->prof_spans.clear();
    for (int g = 0; g < PROF_GROUPS; ++g) { m->prof_ms[g] = 0.f; m->prof_n[g] = 0; }
    m->prof_on = true;
    return ADED_OK;
}

aded_status aded_profile_end(aded_model* m, float* out_ms_host, int32_t* out_launches_host, void* stream) {
    if (!m || !out_ms_host || !out_launches_host) return ADED_ERR_INVALID_ARG;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    m->prof_on = false;
    ADED_CUDA_TRY(cudaStreamSynchronize(st));
    for (ProfSpan& sp : m->prof_spans) {
        float ms = 0.f;
        ADED_CUDA_TRY(cudaEventElapsedTime(&ms, sp.a, sp.b));
        m->prof_ms[sp.group] += ms;
        m->prof_n[sp.group] += sp.launches;
        m->prof_pool.push_back(sp.a);
        m->prof_pool.push_back(sp.b);
    }
    m->prof_spans.clear();
    for (int g = 0; g < PROF_GROUPS; ++g) { out_ms_host[g] = m->prof_ms[g]; out_launches_host[g] = m->prof_n[g]; }
    return ADED_OK;
}

aded_status aded_trace_begin(aded_model* m, void* stream) {
    if (!m) return ADED_ERR_INVALID_ARG;
    const int32_t on_and_count[2] = {1, 0};
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    ADED_CUDA_TRY(cudaMemcpyAsync(m->status + 1, on_and_count, sizeof on_and_count, cudaMemcpyHostToDevice, st));
    ADED_CUDA_TRY(cudaStreamSynchronize(st));     // the two words are a stack variable
    return ADED_OK;
}

aded_status aded_trace_end(aded_model* m, uint64_t* out_ns_host, int32_t* out_kind_host, int32_t max_marks,
                           int32_t* out_n_host, void* stream) {
    if (!m || !out_ns_host || !out_kind_host || !out_n_host || max_marks < 1) return ADED_ERR_INVALID_ARG;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    int32_t words[2] = {0, 0};
    ADED_CUDA_TRY(cudaMemcpyAsync(words, m->status + 1, sizeof words, cudaMemcpyDeviceToHost, st));
    ADED_CUDA_TRY(cudaStreamSynchronize(st));
    const int32_t off = 0;
    ADED_CUDA_TRY(cudaMemcpyAsync(m->status + 1, &off, sizeof off, cudaMemcpyHostToDevice, st));
    const long long taken = words[1];
    long long n = taken < TRACE_CAP ? taken : TRACE_CAP;      // the ring keeps the last TRACE_CAP marks
    if (n > max_marks) n = max_marks;
    std::vector<uint64_t> ts(TRACE_CAP);
    std::vector<int32_t> kind(TRACE_CAP);
    ADED_CUDA_TRY(cudaMemcpyAsync(ts.data(), m->status + 4, TRACE_CAP * sizeof(uint64_t), cudaMemcpyDeviceToHost, st));
    ADED_CUDA_TRY(cudaMemcpyAsync(kind.data(), m->status + 4 + 2 * TRACE_CAP, TRACE_CAP * sizeof(int32_t), cudaMemcpyDeviceToHost, st));
    ADED_CUDA_TRY(cudaStreamSynchronize(st));
    for (long long i = 0; i < n; ++i) {                       // the last n marks, oldest first
        const long long src = (taken - n + i) & (TRACE_CAP - 1);
        out_ns_host[i] = ts[src];
        out_kind_host[i] = kind[src];
    }
    *out_n_host = (int32_t)n;
    return ADED_OK;
}

aded_status aded_debug_wait_timeout(aded_model* m, int32_t which, uint64_t limit_cycles, void* stream) {
    if (!m || which < 0 || which > 1 || limit_cycles < 1 || limit_cycles > (1ull << 32)) return ADED_ERR_INVALID_ARG;
    // the counter the probe polls: a word of the trace area that only ever holds a small count
    const uint32_t* quiet = reinterpret_cast<const uint32_t*>(m->status + 3);
    note_launch();
    ADED_CUDA_TRY(ws_wait_probe(which, (long long)limit_cycles, quiet, m->status, static_cast<cudaStream_t>(stream)));
    return ADED_OK;
}

aded_status aded_debug_attention_kernel(aded_model* m, int32_t which) {
    if (!m || which < 0 || which > 1) return ADED_ERR_INVALID_ARG;
    if (which == 0) { m->att_tc = m->att_tc_ok; return ADED_OK; }
    if (!m->att_mma) return ADED_ERR_UNSUPPORTED;
    m->att_tc = false;
    return ADED_OK;
}

aded_status aded_debug_weight_layout(aded_model* m, int32_t which) {
    if (!m || which < 0 || which > 1) return ADED_ERR_INVALID_ARG;
    if (!m->ws_ready) return ADED_ERR_UNSUPPORTED;
    if (which == 0) {
        if (m->ws_tiled.empty() || !m->ws_tiled[0]) return ADED_ERR_UNSUPPORTED;
        m->ws_use_tiled = true;
        return ADED_OK;
    }
    m->ws_use_tiled = false;
    return ADED_OK;
}

uint64_t aded_launch_count(void) { return g_launches.load(std::memory_order_relaxed); }

aded_status aded_model_poll_status(aded_model* m, aded_status* out_host, void* stream) {
    if (!m || !out_host) return ADED_ERR_INVALID_ARG;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    int32_t v = 0;
    ADED_CUDA_TRY(cudaMemcpyAsync(&v, m->status, sizeof v, cudaMemcpyDeviceToHost, st));
    ADED_CUDA_TRY(cudaStreamSynchronize(st));
    if (v != 0) {
        ADED_CUDA_TRY(cudaMemsetAsync(m->status, 0, sizeof v, st));
        // a pass that gave up in the middle of a projection's tail may have left its meeting counters mid-count
        if (m->ws_ready) {
            ADED_CUDA_TRY(cudaMemsetAsync(m->ws_counters, 0, (size_t)(m->cfg.vocab / 128) * sizeof(uint32_t), st));
            m->ws_epoch = 0;
        }
        ADED_CUDA_TRY(cudaStreamSynchronize(st));
    }
    *out_host = static_cast<aded_status>(v);
    return ADED_OK;
}

const char* aded_status_string(aded_status s) {
    switch (s) {
        case ADED_OK: return "ok";
        case ADED_ERR_INVALID_ARG: return "invalid argument";
        case ADED_ERR_BAD_TREE: return "malformed draft tree";
        case ADED_ERR_KV_CAPACITY: return "KV cache capacity exceeded";
        case ADED_ERR_TABLE_FULL: return "tri-gram store full";
        case ADED_ERR_OOM: return "out of device memory";
        case ADED_ERR_CUDA: return "CUDA runtime error";
        case ADED_ERR_UNSUPPORTED: return "unsupported configuration";
        case ADED_ERR_TIMEOUT: return "device-side wait ran out";
        case ADED_ERR_INTERNAL: return "index check failed inside a kernel (debug build)";
    }
    return "unknown status";
}

}  // extern "C"
