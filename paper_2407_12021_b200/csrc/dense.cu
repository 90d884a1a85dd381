// Row-wise pieces of the Llama-style decoder around the projections: embedding gather, residual
// add + RMSNorm, rotary embedding + K/V write, SwiGLU, per-row greedy choice, and a plain
// shared-memory GEMM used for fp32 models and for shapes the tensor-core path does not take.
//
// Rounding: activations are stored in the model dtype (bf16 models round to nearest even at
// every store below); all sums are fp32.  Kernels that consume a projection read it through
// GemmOut (gemm_out.cuh): either a plain fp32 matrix or per-CTA partial tiles added in CTA order.
// These are the kernels of fp32 models; bf16 models on the tensor-core path use the four-columns-per-thread
// versions in dense_ws.cu.
#include "aded_internal.cuh"

namespace aded {

__device__ __forceinline__ float warp_sum(float v) {
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
    return v;
}

// Sum over the block; every thread receives the total.  `red` holds 32 floats.
__device__ __forceinline__ float block_sum(float v, float* red) {
    v = warp_sum(v);
    const int w = threadIdx.x >> 5, l = threadIdx.x & 31, nw = (blockDim.x + 31) >> 5;
    __syncthreads();
    if (l == 0) red[w] = v;
    __syncthreads();
    float t = l < nw ? red[l] : 0.f;
    return warp_sum(t);
}

template <typename T>
__global__ void k_embed(const T* __restrict__ table, const CallPtrs* __restrict__ call, T* __restrict__ h,
                        int d, const int32_t* status) {
    pdl_enter();
    if (first_thread_of_grid()) trace_mark(status, TK_OTHER);
    if (*status != 0) return;
    const int32_t* __restrict__ tokens = call->tokens;
    const int r = blockIdx.x;
    const T* src = table + (size_t)tokens[r] * d;
    for (int c = threadIdx.x; c < d; c += blockDim.x) h[(size_t)r * d + c] = src[c];
}

// cos/sin of pos * theta^(-2i/hd) for every row, in double, stored as float: the angles reach
// thousands of radians, where float argument reduction would cost several bf16 ulps.
__global__ void k_rope_table(const int32_t* __restrict__ pos, float* __restrict__ cs, float* __restrict__ sn,
                             int half, double theta, const int32_t* status) {
    pdl_enter();
    if (first_thread_of_grid()) trace_mark(status, TK_OTHER);
    if (*status != 0) return;
    const int r = blockIdx.x;
    for (int i = threadIdx.x; i < half; i += blockDim.x) {
        const double inv = pow(theta, -(double)i / (double)half);
        double s, c;
        sincos((double)pos[r] * inv, &s, &c);
        cs[r * half + i] = (float)c;
        sn[r * half + i] = (float)s;
    }
}

// Residual add + RMSNorm:  h = round(h + y) (when y is given), x = round(h * rsqrt(mean(h^2) + eps) * gain).
// Grid (column chunks of 256, rows): each thread owns one column of one row, so the partial tiles of
// y are gathered with full parallelism.  A chunk leaves its sum of squares in `ssq`; the chunk that
// finishes a row last (per-row counter) adds the row's chunk sums in chunk order and writes x for
// the whole row.  The order of every sum is fixed, so the result does not depend on timing.
template <typename T>
__global__ void __launch_bounds__(256) k_add_rmsnorm(T* __restrict__ h, GemmOut y, int has_y, const T* __restrict__ gain,
                                                     T* __restrict__ x, int d, float eps, float* __restrict__ ssq,
                                                     int32_t* __restrict__ row_count, const int32_t* status) {
    pdl_enter();
    if (first_thread_of_grid()) trace_mark(status, TK_NORM);
    if (*status != 0) return;
    __shared__ float red[32];
    __shared__ int s_last;
    const int r = blockIdx.y, c = blockIdx.x * 256 + threadIdx.x;
    float sq = 0.f;
    if (c < d) {
        float v = to_f32(h[(size_t)r * d + c]);
        if (has_y) {
            const float add = y.mode == 0 ? y.y[(size_t)r * d + c] : gemm_out_at(y, y.tiles[c >> 7], r, c & 127);
            const T nv = from_f32<T>(v + add);
            h[(size_t)r * d + c] = nv;
            v = to_f32(nv);
        }
        sq = v * v;
    }
    sq = block_sum(sq, red);
    if (threadIdx.x == 0) {
        ssq[r * 32 + blockIdx.x] = sq;
        __threadfence();
        const int prev = atomicAdd(&row_count[r], 1);
        s_last = prev == (int)gridDim.x - 1;
        if (s_last) row_count[r] = 0;
    }
    __syncthreads();
    if (!s_last) return;
    __threadfence();
    float total = 0.f;
    for (int i = 0; i < (int)gridDim.x; ++i) total += __ldcg(ssq + r * 32 + i);
    const float inv = rsqrtf(total / (float)d + eps);
    if (sizeof(T) == 2) {
        // two columns per access
        const uint32_t* hr = reinterpret_cast<const uint32_t*>(h + (size_t)r * d);
        const uint32_t* gr = reinterpret_cast<const uint32_t*>(gain);
        uint32_t* xr = reinterpret_cast<uint32_t*>(x + (size_t)r * d);
        for (int cc = threadIdx.x; cc < d / 2; cc += 256) {
            const uint32_t hv = __ldcg(hr + cc), gv = gr[cc];
            const __nv_bfloat162 hb = *reinterpret_cast<const __nv_bfloat162*>(&hv);
            const __nv_bfloat162 gb = *reinterpret_cast<const __nv_bfloat162*>(&gv);
            const __nv_bfloat162 o = __floats2bfloat162_rn(__low2float(hb) * inv * __low2float(gb),
                                                           __high2float(hb) * inv * __high2float(gb));
            xr[cc] = *reinterpret_cast<const uint32_t*>(&o);
        }
    } else {
        const float* hr = reinterpret_cast<const float*>(h) + (size_t)r * d;
        for (int cc = threadIdx.x; cc < d; cc += 256)
            x[(size_t)r * d + cc] = from_f32<T>(__ldcg(hr + cc) * inv * to_f32(gain[cc]));
    }
}

// y[r, n] = sum_k x[r, k] * w[n, k]; 64 x 64 output tile per block, 16-wide k slabs in shared
// memory, 4 x 4 outputs per thread, fp32 accumulation in k order.
template <typename T>
__global__ void __launch_bounds__(256) k_gemm_plain(const T* __restrict__ x, const T* __restrict__ w,
                                                    float* __restrict__ y, int rows, int n, int k,
                                                    const int32_t* status, int trace_kind) {
    pdl_enter();
    if (first_thread_of_grid()) trace_mark(status, trace_kind);
    if (*status != 0) return;
    __shared__ float sx[16][64 + 4];
    __shared__ float sw[16][64 + 4];
    const int r0 = blockIdx.y * 64, n0 = blockIdx.x * 64;
    const int tx = threadIdx.x & 15, ty = threadIdx.x >> 4;
    float acc[4][4] = {};
    for (int k0 = 0; k0 < k; k0 += 16) {
        for (int e = threadIdx.x; e < 64 * 16; e += 256) {
            const int rr = e >> 4, kk = e & 15;
            const bool kin = k0 + kk < k;
            sx[kk][rr] = (r0 + rr < rows && kin) ? to_f32(x[(size_t)(r0 + rr) * k + k0 + kk]) : 0.f;
            sw[kk][rr] = (n0 + rr < n && kin) ? to_f32(w[(size_t)(n0 + rr) * k + k0 + kk]) : 0.f;
        }
        __syncthreads();
#pragma unroll
        for (int kk = 0; kk < 16; ++kk) {
            float a[4], b[4];
#pragma unroll
            for (int i = 0; i < 4; ++i) { a[i] = sx[kk][ty * 4 + i]; b[i] = sw[kk][tx * 4 + i]; }
#pragma unroll
            for (int i = 0; i < 4; ++i)
#pragma unroll
                for (int j = 0; j < 4; ++j) acc[i][j] = fmaf(a[i], b[j], acc[i][j]);
        }
        __syncthreads();
    }
#pragma unroll
    for (int i = 0; i < 4; ++i)
#pragma unroll
        for (int j = 0; j < 4; ++j) {
            const int r = r0 + ty * 4 + i, c = n0 + tx * 4 + j;
            if (r < rows && c < n) y[(size_t)r * n + c] = acc[i][j];
        }
}

// Rotary embedding of q and k (pairs (i, i + hd/2), angle from the table), then q -> q buffer and
// k, v -> the cache at slot committed length + local node index.  Block = (row, head).
template <typename T>
__global__ void k_rope_kv(GemmOut qkv, const float* __restrict__ cs, const float* __restrict__ sn,
                          T* __restrict__ q, char* const* __restrict__ base, const int32_t* __restrict__ cap,
                          const int32_t* __restrict__ len, const int32_t* __restrict__ row_seq,
                          const int32_t* __restrict__ row_local, int layer, int H, int hd, const int32_t* status) {
    pdl_enter();
    if (first_thread_of_grid()) trace_mark(status, TK_ROPE);
    if (*status != 0) return;
    const int r = blockIdx.x, hh = blockIdx.y, half = hd >> 1, d = H * hd;
    const int b = row_seq[r];
    const size_t slot = (size_t)len[b] + row_local[r];
    const size_t cp = cap[b];
    T* kdst = reinterpret_cast<T*>(base[b]) + ((((size_t)layer * 2 + 0) * H + hh) * cp + slot) * hd;
    T* vdst = reinterpret_cast<T*>(base[b]) + ((((size_t)layer * 2 + 1) * H + hh) * cp + slot) * hd;
    // the head's q, k and v columns each lie inside one 128-column tile of the projection result
    const int cq = hh * hd, ck = d + hh * hd, cv = 2 * d + hh * hd;
    TileRef tq = {0, 0}, tk = {0, 0}, tv = {0, 0};
    if (qkv.mode == 1) { tq = qkv.tiles[cq >> 7]; tk = qkv.tiles[ck >> 7]; tv = qkv.tiles[cv >> 7]; }
    auto at = [&](const TileRef& t, int col) {
        return qkv.mode == 0 ? qkv.y[(size_t)r * 3 * d + col] : gemm_out_at(qkv, t, r, col & 127);
    };
    for (int i = threadIdx.x; i < half; i += blockDim.x) {
        const float c = cs[r * half + i], s = sn[r * half + i];
        const float q0 = at(tq, cq + i), q1 = at(tq, cq + i + half);
        const float k0 = at(tk, ck + i), k1 = at(tk, ck + i + half);
        q[(size_t)r * d + hh * hd + i] = from_f32<T>(q0 * c - q1 * s);
        q[(size_t)r * d + hh * hd + i + half] = from_f32<T>(q1 * c + q0 * s);
        kdst[i] = from_f32<T>(k0 * c - k1 * s);
        kdst[i + half] = from_f32<T>(k1 * c + k0 * s);
        vdst[i] = from_f32<T>(at(tv, cv + i));
        vdst[i + half] = from_f32<T>(at(tv, cv + i + half));
    }
}

// act = round(silu(gate) * up), gate = gu[:, :F], up = gu[:, F:].
template <typename T>
__global__ void k_swiglu(GemmOut gu, T* __restrict__ act, int F, const int32_t* status) {
    pdl_enter();
    if (first_thread_of_grid()) trace_mark(status, TK_SWIGLU);
    if (*status != 0) return;
    const int r = blockIdx.y;
    const int c = blockIdx.x * blockDim.x + threadIdx.x;
    if (c >= F) return;
    const float g = gemm_out_load(gu, r, c), u = gemm_out_load(gu, r, F + c);
    act[(size_t)r * F + c] = from_f32<T>(g / (1.f + expf(-g)) * u);
}

// Greedy choice per row: largest fp32 logit, lowest index among equals.  Stage 1: grid (chunks, rows),
// every block scans `chunk` columns of one row and leaves (value, index) of its best; stage 2 (one
// thread per row) takes the best of the chunks in ascending column order.
__global__ void __launch_bounds__(256) k_argmax_chunks(GemmOut logits, float* __restrict__ pv, int32_t* __restrict__ pi,
                                                       int V, int chunk, const int32_t* status) {
    pdl_enter();
    if (first_thread_of_grid()) trace_mark(status, TK_PICK);
    if (*status != 0) return;
    __shared__ float sv[8];
    __shared__ int si[8];
    const int r = blockIdx.y;
    const int c0 = blockIdx.x * chunk, c1 = min(V, c0 + chunk);
    float bv = -INFINITY;
    int bi = 0x7fffffff;
    if (logits.mode == 1 && (V & 3) == 0) {
        // partial tiles: four adjacent columns per thread and step, all contributors fetched at once
        for (int c = c0 + threadIdx.x * 4; c < c1; c += 1024) {
            const float4 v = gemm_out_at4(logits, logits.tiles[c >> 7], r, c & 127);
            if (v.x > bv) { bv = v.x; bi = c; }       // columns ascend per thread: first maximum kept
            if (v.y > bv) { bv = v.y; bi = c + 1; }
            if (v.z > bv) { bv = v.z; bi = c + 2; }
            if (v.w > bv) { bv = v.w; bi = c + 3; }
        }
    } else {
        for (int c = c0 + threadIdx.x; c < c1; c += 256) {
            const float v = gemm_out_load(logits, r, c);
            if (v > bv) { bv = v; bi = c; }   // c ascends per thread: first maximum kept
        }
    }
    for (int o = 16; o > 0; o >>= 1) {
        const float ov = __shfl_xor_sync(0xffffffffu, bv, o);
        const int oi = __shfl_xor_sync(0xffffffffu, bi, o);
        if (ov > bv || (ov == bv && oi < bi)) { bv = ov; bi = oi; }
    }
    const int w = threadIdx.x >> 5, l = threadIdx.x & 31;
    if (l == 0) { sv[w] = bv; si[w] = bi; }
    __syncthreads();
    if (threadIdx.x == 0) {
        for (int i = 1; i < 8; ++i)
            if (sv[i] > bv || (sv[i] == bv && si[i] < bi)) { bv = sv[i]; bi = si[i]; }
        pv[r * gridDim.x + blockIdx.x] = bv;
        pi[r * gridDim.x + blockIdx.x] = bi;
    }
}

__global__ void k_argmax_final(const float* __restrict__ pv, const int32_t* __restrict__ pi, int32_t* __restrict__ best,
                               int chunks, int rows, const int32_t* status) {
    pdl_enter();
    if (first_thread_of_grid()) trace_mark(status, TK_PICK);
    if (*status != 0) return;
    const int r = blockIdx.x * blockDim.x + threadIdx.x;
    if (r >= rows) return;
    float bv = -INFINITY;
    int bi = 0x7fffffff;
    for (int i = 0; i < chunks; ++i) {
        const float v = pv[r * chunks + i];
        const int idx = pi[r * chunks + i];
        if (v > bv || (v == bv && idx < bi)) { bv = v; bi = idx; }
    }
    best[r] = bi == 0x7fffffff ? 0 : bi;
}

__global__ void k_materialize(GemmOut src, float* __restrict__ dst, int n, const int32_t* status) {
    pdl_enter();
    if (first_thread_of_grid()) trace_mark(status, TK_OTHER);
    if (*status != 0) return;
    const int r = blockIdx.y;
    const int c = blockIdx.x * blockDim.x + threadIdx.x;
    if (c < n) dst[(size_t)r * n + c] = gemm_out_load(src, r, c);
}

// ---- launchers --------------------------------------------------------------------------
#define BY_DTYPE(m, CALL_BF16, CALL_F32) \
    do { if ((m)->cfg.dtype == ADED_BF16) { CALL_BF16; } else { CALL_F32; } } while (0)

void launch_embed(aded_model* m, int rows, cudaStream_t st) {
    const int d = m->cfg.d_model;
    BY_DTYPE(m, (launch_k(k_embed<bf16>, rows, 256, 0, st, (const bf16*)m->top.embed, m->call_dev, (bf16*)m->h, d, m->status)),
             (launch_k(k_embed<float>, rows, 256, 0, st, (const float*)m->top.embed, m->call_dev, (float*)m->h, d, m->status)));
}

void launch_rope_table(aded_model* m, int rows, cudaStream_t st) {
    launch_k(k_rope_table, rows, 64, 0, st, m->rows.pos, m->rope_cos, m->rope_sin, m->cfg.head_dim / 2,
                                      (double)m->cfg.rope_theta, m->status);
}

void launch_add_rmsnorm(aded_model* m, const GemmOut* y, const void* gain, int rows, cudaStream_t st) {
    const int d = m->cfg.d_model;
    if (y && y->mode == 1 && m->cfg.dtype == ADED_BF16) { launch_add_rmsnorm_ws(m, *y, gain, rows, st); return; }
    GemmOut none = {};
    const GemmOut& yy = y ? *y : none;
    const int has = y != nullptr;
    dim3 grid((d + 255) / 256, rows);
    BY_DTYPE(m, (launch_k(k_add_rmsnorm<bf16>, grid, 256, 0, st, (bf16*)m->h, yy, has, (const bf16*)gain, (bf16*)m->x, d, m->cfg.rms_eps, m->norm_ssq, m->norm_count, m->status)),
             (launch_k(k_add_rmsnorm<float>, grid, 256, 0, st, (float*)m->h, yy, has, (const float*)gain, (float*)m->x, d, m->cfg.rms_eps, m->norm_ssq, m->norm_count, m->status)));
}

static void launch_gemm_plain(aded_model* m, const void* x, const void* w, float* y, int rows, int n, int k, int trace_kind,
                              cudaStream_t st) {
    dim3 grid((n + 63) / 64, (rows + 63) / 64);
    BY_DTYPE(m, (launch_k(k_gemm_plain<bf16>, grid, 256, 0, st, (const bf16*)x, (const bf16*)w, y, rows, n, k, m->status, trace_kind)),
             (launch_k(k_gemm_plain<float>, grid, 256, 0, st, (const float*)x, (const float*)w, y, rows, n, k, m->status, trace_kind)));
}

GemmOut launch_gemm(aded_model* m, int w_map, int x_map, const void* x, const void* w, float* y, int rows, int n, int k,
                    int epi_mode, int trace_kind, cudaStream_t st) {
    GemmOut out = {};
    out.n = n;
    out.rows = rows;
    if (m->ws_ready && w_map >= 0 && x_map >= 0 && ws_supported(n, k)) {
        // tensor-core path, up to 128 (or 256) rows of x per pass over the weights; the result stays in slots
        const int table = w_map < 4 * m->cfg.n_layers ? w_map % 4 : 4;
        WsEpilogue e = {};
        e.mode = epi_mode;
        e.tiles = m->ws_tiles[table];
        e.counters = m->ws_counters;
        e.cand_val = m->cand_val;
        e.cand_idx = m->cand_idx;
        // a pass takes 128 rows; calls with more rows (ragged batches) use 256-row passes: half as many trips over W
        const int blk = rows > 128 ? 256 : 128;
        for (int row0 = 0; row0 < rows; row0 += blk) {
            const int part = rows - row0 < blk ? rows - row0 : blk;
            if (epi_mode != WS_EPI_SLOTS) e.epoch = ++m->ws_epoch;
            ws_launch(m->ws_maps[w_map], m->ws_use_tiled ? m->ws_tiled[w_map] : nullptr, m->ws_maps[x_map], m->ws_maps[x_map + 3], part, row0, blk, n, k, m->ws_slots, m->status, e, trace_kind, m->device, m->ws_one_per_sm[table], st);
        }
        out.blk_shift = blk == 256 ? 8 : 7;
        out.mode = 1;
        out.slots = m->ws_slots;
        out.n_tiles = n / 128;
        out.kb = k / 64;
        out.g = ws_grid(m->device, n, k, m->ws_one_per_sm[table]);
        out.tiles = m->ws_tiles[table];
        return out;
    }
    launch_gemm_plain(m, x, w, y, rows, n, k, trace_kind, st);
    out.mode = 0;
    out.y = y;
    return out;
}

void launch_materialize(aded_model* m, const GemmOut& src, float* dst, int rows, cudaStream_t st) {
    dim3 grid((src.n + 255) / 256, rows);
    launch_k(k_materialize, grid, 256, 0, st, src, dst, src.n, m->status);
}

void launch_rope_kv(aded_model* m, aded_kv* kv, const GemmOut& qkv, int layer, int rows, cudaStream_t st) {
    if (qkv.mode == 1 && m->cfg.dtype == ADED_BF16) { launch_rope_kv_ws(m, kv, qkv, layer, rows, st); return; }
    dim3 grid(rows, m->cfg.n_heads);
    const int H = m->cfg.n_heads, hd = m->cfg.head_dim;
    BY_DTYPE(m, (launch_k(k_rope_kv<bf16>, grid, 64, 0, st, qkv, m->rope_cos, m->rope_sin, (bf16*)m->q, kv->base_dev, kv->cap_dev, kv->len_dev, m->rows.seq, m->rows.local, layer, H, hd, m->status)),
             (launch_k(k_rope_kv<float>, grid, 64, 0, st, qkv, m->rope_cos, m->rope_sin, (float*)m->q, kv->base_dev, kv->cap_dev, kv->len_dev, m->rows.seq, m->rows.local, layer, H, hd, m->status)));
}

void launch_swiglu(aded_model* m, const GemmOut& gu, int rows, cudaStream_t st) {
    if (gu.mode == 1 && m->cfg.dtype == ADED_BF16) { launch_swiglu_ws(m, gu, rows, st); return; }
    const int F = m->cfg.d_ffn;
    dim3 grid((F + 255) / 256, rows);
    BY_DTYPE(m, (launch_k(k_swiglu<bf16>, grid, 256, 0, st, gu, (bf16*)m->act, F, m->status)),
             (launch_k(k_swiglu<float>, grid, 256, 0, st, gu, (float*)m->act, F, m->status)));
}

void launch_argmax(aded_model* m, const GemmOut& logits, int rows, cudaStream_t st) {
    const int V = m->cfg.vocab;
    const int chunks = ARGMAX_CHUNKS;
    const int chunk = ((V + chunks - 1) / chunks + 127) / 128 * 128;   // whole 128-column tiles per block
    dim3 grid(chunks, rows);
    launch_k(k_argmax_chunks, grid, 256, 0, st, logits, m->argmax_val, m->argmax_idx, V, chunk, m->status);
    launch_k(k_argmax_final, (rows + 127) / 128, 128, 0, st, m->argmax_val, m->argmax_idx, m->best, chunks, rows, m->status);
}

}  // namespace aded
