// bf16 consumers of the tensor-core GEMM's partial tiles, four columns per thread.
//
// Same arithmetic as the generic kernels in dense.cu (residual add + RMSNorm, rotary + K/V write,
// SwiGLU), specialised for the case that matters for speed: the projection result lives in slots
// (gemm_out.cuh) and the model is bf16.  Each thread gathers four adjacent columns of every
// contributing slot with 16-byte loads that are all in flight at once, so a kernel is one or two
// memory round trips deep instead of one per contributor.  Also here: embedding lookup + first
// RMSNorm, and the greedy choice + approval walk that follows the LM head's per-tile candidates.
#include "aded_internal.cuh"

namespace aded {

__device__ __forceinline__ float warp_sum_f(float v) {
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
    return v;
}

// Embedding lookup + the first layer's RMSNorm in one kernel (bf16): h = embed[token], x = norm(h).
// One block of 1024 threads per row, four columns per thread and pass, as k_add_rmsnorm_ws.
__global__ void __launch_bounds__(1024) k_embed_norm_ws(const bf16* __restrict__ table, const CallPtrs* __restrict__ call,
                                                        bf16* __restrict__ h, const bf16* __restrict__ gain, bf16* __restrict__ x,
                                                        int d, int vocab, float eps, const int32_t* status) {
    pdl_launch_dependents();
    __shared__ float red[32];
    const int r = blockIdx.x;
    float4 gv[2];
#pragma unroll
    for (int i = 0; i < 2; ++i) {
        const int c = (i * 1024 + threadIdx.x) * 4;
        if (c < d) gv[i] = unpack4_bf16(*reinterpret_cast<const uint2*>(gain + c));
    }
    pdl_wait();
    if (first_thread_of_grid()) trace_mark(status, TK_OTHER);
    const int pass_status = *status;
    int tok = call->tokens[r];
    if (tok < 0 || tok >= vocab) tok = 0;          // a token outside the vocabulary has been reported by the tree check
    const bf16* src = table + (size_t)tok * d;
    float4 v[2];
    float sq = 0.f;
#pragma unroll
    for (int i = 0; i < 2; ++i) {
        const int c = (i * 1024 + threadIdx.x) * 4;
        if (c < d) {
            const uint2 raw = *reinterpret_cast<const uint2*>(src + c);
            if (pass_status == 0) *reinterpret_cast<uint2*>(h + (size_t)r * d + c) = raw;
            v[i] = unpack4_bf16(raw);
            sq += v[i].x * v[i].x + v[i].y * v[i].y + v[i].z * v[i].z + v[i].w * v[i].w;
        }
    }
    sq = warp_sum_f(sq);
    if ((threadIdx.x & 31) == 0) red[threadIdx.x >> 5] = sq;
    __syncthreads();
    float total = 0.f;
#pragma unroll
    for (int i = 0; i < 32; ++i) total += red[i];
    const float inv = rsqrtf(total / (float)d + eps);
    if (pass_status != 0) return;
#pragma unroll
    for (int i = 0; i < 2; ++i) {
        const int c = (i * 1024 + threadIdx.x) * 4;
        if (c < d)
            *reinterpret_cast<uint2*>(x + (size_t)r * d + c) =
                pack4_bf16(v[i].x * inv * gv[i].x, v[i].y * inv * gv[i].y, v[i].z * inv * gv[i].z, v[i].w * inv * gv[i].w);
    }
}

// Greedy token of every row from the LM head's per-tile candidates (largest value, lowest column among
// equals -- a tile's candidate already is its lowest best column), then the approval walk of tree.cu.
// One block of 1024 threads per sequence; a warp per row, every lane's candidates fetched at once.
constexpr int PICK_THREADS = 1024, PICK_PER_LANE = 8;
__global__ void __launch_bounds__(PICK_THREADS) k_pick_accept(const CallPtrs* __restrict__ call, const float* __restrict__ cand_val,
                                                              const int32_t* __restrict__ cand_idx, int n_tiles,
                                                              const int32_t* __restrict__ row_off, int32_t* __restrict__ best,
                                                              const int32_t* __restrict__ depth, const int32_t* __restrict__ len,
                                                              int32_t* __restrict__ path, int32_t* __restrict__ new_len,
                                                              const int32_t* status) {
    pdl_enter();
    if (first_thread_of_grid()) trace_mark(status, TK_PICK);
    __shared__ int32_t s_par[ADED_MAX_NODES], s_tok[ADED_MAX_NODES], s_best[ADED_MAX_NODES], s_dep[ADED_MAX_NODES];
    const int b = blockIdx.x;
    const int pass_status = *status;
    const int off = row_off[b];
    const int T = min(row_off[b + 1] - off, (int)ADED_MAX_NODES);
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    for (int i = warp; i < T; i += PICK_THREADS / 32) {
        float bv = -INFINITY;
        int bi = 0x7fffffff;
        const float* pv = cand_val + (size_t)(off + i) * n_tiles;
        const int32_t* pi = cand_idx + (size_t)(off + i) * n_tiles;
        for (int t0 = 0; t0 < n_tiles; t0 += 32 * PICK_PER_LANE) {
            float v[PICK_PER_LANE];
            int idx[PICK_PER_LANE];
#pragma unroll
            for (int j = 0; j < PICK_PER_LANE; ++j) {
                const int t = t0 + j * 32 + lane;
                v[j] = t < n_tiles ? __ldcg(pv + t) : -INFINITY;
                idx[j] = t < n_tiles ? __ldcg(pi + t) : 0x7fffffff;
            }
#pragma unroll
            for (int j = 0; j < PICK_PER_LANE; ++j)
                if (v[j] > bv || (v[j] == bv && idx[j] < bi)) { bv = v[j]; bi = idx[j]; }
        }
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) {
            const float ov = __shfl_xor_sync(0xffffffffu, bv, o);
            const int oi = __shfl_xor_sync(0xffffffffu, bi, o);
            if (ov > bv || (ov == bv && oi < bi)) { bv = ov; bi = oi; }
        }
        if (lane == 0) {
            const int pick = bi == 0x7fffffff ? 0 : bi;
            s_best[i] = pick;
            if (pass_status == 0) best[off + i] = pick;
        }
    }
    for (int i = threadIdx.x; i < T; i += blockDim.x) {
        s_par[i] = call->parents[off + i];
        s_tok[i] = call->tokens[off + i];
        s_dep[i] = depth[off + i];
    }
    __syncthreads();
    if (threadIdx.x == 0)
        approval_walk(s_par, s_tok, s_best, s_dep, T, pass_status, len[b], call->out_tokens + (size_t)b * call->out_stride,
                      call->out_len + b, path + b * ADED_MAX_NODES, new_len + b);
}

// Residual add + RMSNorm (see k_add_rmsnorm): one block of 1024 threads per row, four columns per
// thread and pass (two passes cover d up to 8192).  The row stays in registers between the sum of
// squares and the scaling, so the kernel is: gather the projection's slots, one block reduction,
// store h and x.  The contributor table and the gain are not written by any kernel of the pass and
// are fetched before waiting for the previous kernel.
// The next kernel (a projection) is released right after the wait, not at the top of the kernel.  Measured on
// a 32-layer step: released at the top (its blocks can then appear while the previous projection is still
// running) the step is 1.3 % slower; released after the gather or at exit (its weight prefetch no longer
// runs under this kernel) 4 % slower.  The SwiGLU and rotary kernels below do the same (for them the top of
// the kernel measures the same; the difference comes from this kernel, whose blocks each take a whole SM's registers).
__global__ void __launch_bounds__(1024) k_add_rmsnorm_ws(bf16* __restrict__ h, GemmOut y, const bf16* __restrict__ gain,
                                                         bf16* __restrict__ x, int d, float eps, const int32_t* status) {
    __shared__ float red[32];
    const int r = blockIdx.x;
    TileRef tr[2];
    float4 gv[2];
#pragma unroll
    for (int i = 0; i < 2; ++i) {
        const int c = (i * 1024 + threadIdx.x) * 4;
        if (c < d) {
            tr[i] = y.tiles[c >> 7];
            gv[i] = unpack4_bf16(*reinterpret_cast<const uint2*>(gain + c));
        }
    }
    pdl_wait();
    pdl_launch_dependents();
    if (first_thread_of_grid()) trace_mark(status, TK_NORM);
    const int pass_status = *status;     // acted on before the first store; the loads below are valid in any case
    float4 v[2];
    float sq = 0.f;
#pragma unroll
    for (int i = 0; i < 2; ++i) {
        const int c = (i * 1024 + threadIdx.x) * 4;
        if (c < d) {
            uint2* hp = reinterpret_cast<uint2*>(h + (size_t)r * d + c);
            const float4 hv = unpack4_bf16(*hp);
            if (!ADED_IN_RANGE(tr[i].first_slot >= 0 && tr[i].first_slot + tr[i].count <= y.n_tiles + y.g, status)) tr[i].count = 0;
            const float4 add = gemm_out_at4(y, tr[i], r, c & 127);
            const uint2 nv = pack4_bf16(hv.x + add.x, hv.y + add.y, hv.z + add.z, hv.w + add.w);
            if (pass_status == 0) *hp = nv;
            v[i] = unpack4_bf16(nv);
            sq += v[i].x * v[i].x + v[i].y * v[i].y + v[i].z * v[i].z + v[i].w * v[i].w;
        }
    }
    sq = warp_sum_f(sq);
    if ((threadIdx.x & 31) == 0) red[threadIdx.x >> 5] = sq;
    __syncthreads();
    float total = 0.f;
#pragma unroll
    for (int i = 0; i < 32; ++i) total += red[i];      // same order in every thread
    const float inv = rsqrtf(total / (float)d + eps);
    if (pass_status != 0) return;
#pragma unroll
    for (int i = 0; i < 2; ++i) {
        const int c = (i * 1024 + threadIdx.x) * 4;
        if (c < d)
            *reinterpret_cast<uint2*>(x + (size_t)r * d + c) =
                pack4_bf16(v[i].x * inv * gv[i].x, v[i].y * inv * gv[i].y, v[i].z * inv * gv[i].z, v[i].w * inv * gv[i].w);
    }
}

// act = round(silu(gate) * up): grid (chunks of 1024 columns, rows), four columns per thread.
__global__ void __launch_bounds__(256) k_swiglu_ws(GemmOut gu, bf16* __restrict__ act, int F, const int32_t* status) {
    const int r = blockIdx.y, c = (blockIdx.x * 256 + threadIdx.x) * 4;
    TileRef tg = {0, 0}, tu = {0, 0};
    if (c < F) { tg = gu.tiles[c >> 7]; tu = gu.tiles[(F + c) >> 7]; }   // the table is constant: read it before waiting
    pdl_wait();
    pdl_launch_dependents();
    if (first_thread_of_grid()) trace_mark(status, TK_SWIGLU);
    if (c >= F) return;
    const int pass_status = *status;     // checked before the store, not before the loads
    if (!ADED_IN_RANGE(tg.first_slot + tg.count <= gu.n_tiles + gu.g && tu.first_slot + tu.count <= gu.n_tiles + gu.g, status)) return;
    float4 g, u;
    constexpr int SB = 4;      // gate/up tiles have two or three contributors at the 7B and 13B widths
    if (tg.count <= SB && tu.count <= SB) {
        float4 fg[SB], fu[SB];
        gemm_out_fetch4<SB>(gu, tg, r, c & 127, fg);
        gemm_out_fetch4<SB>(gu, tu, r, (F + c) & 127, fu);
        g = gemm_out_sum4<SB>(fg, tg);
        u = gemm_out_sum4<SB>(fu, tu);
    } else {
        g = gemm_out_at4(gu, tg, r, c & 127);
        u = gemm_out_at4(gu, tu, r, (F + c) & 127);
    }
    if (pass_status != 0) return;
    *reinterpret_cast<uint2*>(act + (size_t)r * F + c) = swiglu4(g, u);
}

// Rotary embedding + K/V write (see k_rope_kv): hd/8 threads per (row, head), each owning four adjacent
// rotary pairs (i .. i+3, i+half .. i+half+3); a block of ROPE_WS_THREADS threads takes consecutive heads
// of one row, so its warps are full and a pass is a few hundred blocks instead of rows x heads tiny ones.
constexpr int ROPE_WS_THREADS = 128;
__global__ void __launch_bounds__(ROPE_WS_THREADS)
k_rope_kv_ws(GemmOut qkv, const float* __restrict__ cs, const float* __restrict__ sn,
             bf16* __restrict__ q, char* const* __restrict__ base, const int32_t* __restrict__ cap,
             const int32_t* __restrict__ len, const int32_t* __restrict__ row_seq,
             const int32_t* __restrict__ row_local, int layer, int H, int hd, const int32_t* status) {
    const int tph = hd >> 3;                                   // threads per head
    const int r = blockIdx.x, half = hd >> 1, d = H * hd;
    const int hh = blockIdx.y * (ROPE_WS_THREADS / tph) + threadIdx.x / tph;
    const int i = (threadIdx.x % tph) * 4;
    const bool mine = hh < H;
    const int hc = mine ? hh : 0;
    const int cq = hc * hd, ck = d + hc * hd, cv = 2 * d + hc * hd;
    const TileRef tq = qkv.tiles[cq >> 7], tk = qkv.tiles[ck >> 7], tv = qkv.tiles[cv >> 7];   // constant table
    pdl_wait();
    pdl_launch_dependents();
    if (first_thread_of_grid()) trace_mark(status, TK_ROPE);
    if (!mine) return;
    const int pass_status = *status;     // checked before the stores, not before the loads
    const int b = row_seq[r];
    const size_t slot = (size_t)len[b] + row_local[r];
    const size_t cp = cap[b];
    bf16* kdst = reinterpret_cast<bf16*>(base[b]) + ((((size_t)layer * 2 + 0) * H + hh) * cp + slot) * hd;
    bf16* vdst = reinterpret_cast<bf16*>(base[b]) + ((((size_t)layer * 2 + 1) * H + hh) * cp + slot) * hd;
    const bool in_range = ADED_IN_RANGE(slot < cp && tq.first_slot + tq.count <= qkv.n_tiles + qkv.g && tv.first_slot + tv.count <= qkv.n_tiles + qkv.g, status);
    rope_kv_item(qkv, tq, tk, tv, r, cq, ck, cv, i, half, cs + r * half, sn + r * half, q + (size_t)r * d + hh * hd, kdst, vdst,
                 pass_status == 0 && in_range);
}

// ---- launchers (callers have checked: bf16 model, tensor-core path) ----------------------------
bool embed_norm_ws_supported(const aded_model* m) {
    return m->cfg.dtype == ADED_BF16 && m->cfg.d_model % 4 == 0 && m->cfg.d_model <= 8192;
}

void launch_embed_norm_ws(aded_model* m, const void* gain, int rows, cudaStream_t st) {
    launch_k(k_embed_norm_ws, dim3(rows), dim3(1024), 0, st, (const bf16*)m->top.embed, (const CallPtrs*)m->call_dev, (bf16*)m->h,
             (const bf16*)gain, (bf16*)m->x, m->cfg.d_model, m->cfg.vocab, m->cfg.rms_eps, (const int32_t*)m->status);
}

void launch_pick_accept(aded_model* m, aded_kv* kv, int batch, int n_tiles, cudaStream_t st) {
    launch_k(k_pick_accept, dim3(batch), dim3(PICK_THREADS), 0, st, (const CallPtrs*)m->call_dev, (const float*)m->cand_val,
             (const int32_t*)m->cand_idx, n_tiles, (const int32_t*)m->seqs.row_off, m->best, (const int32_t*)m->rows.depth,
             (const int32_t*)kv->len_dev, m->seqs.path, m->seqs.new_len, (const int32_t*)m->status);
}

void launch_add_rmsnorm_ws(aded_model* m, const GemmOut& y, const void* gain, int rows, cudaStream_t st) {
    const int d = m->cfg.d_model;
    launch_k(k_add_rmsnorm_ws, dim3(rows), dim3(1024), 0, st, (bf16*)m->h, y, (const bf16*)gain, (bf16*)m->x, d, m->cfg.rms_eps,
             (const int32_t*)m->status);
}

void launch_swiglu_ws(aded_model* m, const GemmOut& gu, int rows, cudaStream_t st) {
    const int F = m->cfg.d_ffn;
    dim3 grid((F + 1023) / 1024, rows);
    launch_k(k_swiglu_ws, grid, dim3(256), 0, st, gu, (bf16*)m->act, F, (const int32_t*)m->status);
}

void launch_rope_kv_ws(aded_model* m, aded_kv* kv, const GemmOut& qkv, int layer, int rows, cudaStream_t st) {
    const int heads_per_block = ROPE_WS_THREADS / (m->cfg.head_dim / 8);
    dim3 grid(rows, (m->cfg.n_heads + heads_per_block - 1) / heads_per_block);
    launch_k(k_rope_kv_ws, grid, dim3(ROPE_WS_THREADS), 0, st, qkv, (const float*)m->rope_cos, (const float*)m->rope_sin, (bf16*)m->q,
             (char* const*)kv->base_dev, (const int32_t*)kv->cap_dev, (const int32_t*)kv->len_dev,
             (const int32_t*)m->rows.seq, (const int32_t*)m->rows.local, layer, m->cfg.n_heads, m->cfg.head_dim,
             (const int32_t*)m->status);
}

}  // namespace aded
