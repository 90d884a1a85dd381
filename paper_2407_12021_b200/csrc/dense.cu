// Row-wise pieces of the Llama-style decoder around the projections: embedding gather, RMSNorm,
// residual add, rotary embedding + K/V write, SwiGLU, per-row greedy choice, and a plain
// shared-memory GEMM used for fp32 models and for shapes the tensor-core path does not take.
//
// Rounding: activations are stored in the model dtype (bf16 models round to nearest even at
// every store below); all sums are fp32.
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
__global__ void k_embed(const T* __restrict__ table, const int32_t* __restrict__ tokens, T* __restrict__ h,
                        int d, const int32_t* status) {
    if (*status != 0) return;
    const int r = blockIdx.x;
    const T* src = table + (size_t)tokens[r] * d;
    for (int c = threadIdx.x; c < d; c += blockDim.x) h[(size_t)r * d + c] = src[c];
}

// cos/sin of pos * theta^(-2i/hd) for every row, in double, stored as float: the angles reach
// thousands of radians, where float argument reduction would cost several bf16 ulps.
__global__ void k_rope_table(const int32_t* __restrict__ pos, float* __restrict__ cs, float* __restrict__ sn,
                             int half, double theta, const int32_t* status) {
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

// x = round(h * rsqrt(mean(h^2) + eps) * gain); when `y` is given, first h = round(h + y).
template <typename T>
__global__ void k_add_rmsnorm(T* __restrict__ h, GemmOut y, int has_y, const T* __restrict__ gain,
                              T* __restrict__ x, int d, float eps, const int32_t* status) {
    if (*status != 0) return;
    __shared__ float red[32];
    __shared__ TileRef tiles[64];          // contributors of each 128-column tile of y (d <= 8192)
    const int r = blockIdx.x;
    if (has_y && y.mode == 1) {
        for (int t = threadIdx.x; t < y.n_tiles; t += blockDim.x) tiles[t] = gemm_tile_ref(y, t);
        __syncthreads();
    }
    T* hr = h + (size_t)r * d;
    float ss = 0.f;
    for (int c = threadIdx.x; c < d; c += blockDim.x) {
        float v = to_f32(hr[c]);
        if (has_y) {
            const float add = y.mode == 0 ? y.y[(size_t)r * d + c] : gemm_out_at(y, tiles[c >> 7], r, c & 127);
            const T nv = from_f32<T>(v + add);
            hr[c] = nv;
            v = to_f32(nv);
        }
        ss += v * v;
    }
    ss = block_sum(ss, red);
    const float inv = rsqrtf(ss / (float)d + eps);
    for (int c = threadIdx.x; c < d; c += blockDim.x)
        x[(size_t)r * d + c] = from_f32<T>(to_f32(hr[c]) * inv * to_f32(gain[c]));
}

// y[r, n] = sum_k x[r, k] * w[n, k]; 64 x 64 output tile per block, 16-wide k slabs in shared
// memory, 4 x 4 outputs per thread, fp32 accumulation in k order.
template <typename T>
__global__ void __launch_bounds__(256) k_gemm_plain(const T* __restrict__ x, const T* __restrict__ w,
                                                    float* __restrict__ y, int rows, int n, int k,
                                                    const int32_t* status) {
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
    if (qkv.mode == 1) { tq = gemm_tile_ref(qkv, cq >> 7); tk = gemm_tile_ref(qkv, ck >> 7); tv = gemm_tile_ref(qkv, cv >> 7); }
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
    if (*status != 0) return;
    const int r = blockIdx.y;
    const int c = blockIdx.x * blockDim.x + threadIdx.x;
    if (c >= F) return;
    const float g = gemm_out_load(gu, r, c), u = gemm_out_load(gu, r, F + c);
    act[(size_t)r * F + c] = from_f32<T>(g / (1.f + expf(-g)) * u);
}

// Greedy choice per row: largest fp32 logit, lowest index among equals.
__global__ void k_argmax(GemmOut logits, int32_t* __restrict__ best, int V, const int32_t* status) {
    if (*status != 0) return;
    __shared__ float sv[32];
    __shared__ int si[32];
    extern __shared__ TileRef tiles[];     // contributors of each 128-column tile (tensor-core path)
    const int r = blockIdx.x;
    if (logits.mode == 1) {
        for (int t = threadIdx.x; t < logits.n_tiles; t += blockDim.x) tiles[t] = gemm_tile_ref(logits, t);
        __syncthreads();
    }
    float bv = -INFINITY;
    int bi = 0x7fffffff;
    for (int c = threadIdx.x; c < V; c += blockDim.x) {
        const float v = logits.mode == 0 ? logits.y[(size_t)r * V + c] : gemm_out_at(logits, tiles[c >> 7], r, c & 127);
        if (v > bv) { bv = v; bi = c; }   // c ascends per thread: first maximum kept
    }
    for (int o = 16; o > 0; o >>= 1) {
        const float ov = __shfl_xor_sync(0xffffffffu, bv, o);
        const int oi = __shfl_xor_sync(0xffffffffu, bi, o);
        if (ov > bv || (ov == bv && oi < bi)) { bv = ov; bi = oi; }
    }
    const int w = threadIdx.x >> 5, l = threadIdx.x & 31;
    if (l == 0) { sv[w] = bv; si[w] = bi; }
    __syncthreads();
    if (w == 0) {
        const int nw = blockDim.x >> 5;
        bv = l < nw ? sv[l] : -INFINITY;
        bi = l < nw ? si[l] : 0x7fffffff;
        for (int o = 16; o > 0; o >>= 1) {
            const float ov = __shfl_xor_sync(0xffffffffu, bv, o);
            const int oi = __shfl_xor_sync(0xffffffffu, bi, o);
            if (ov > bv || (ov == bv && oi < bi)) { bv = ov; bi = oi; }
        }
        if (l == 0) best[r] = bi == 0x7fffffff ? 0 : bi;
    }
}

__global__ void k_materialize(GemmOut src, float* __restrict__ dst, int n, const int32_t* status) {
    if (*status != 0) return;
    const int r = blockIdx.y;
    const int c = blockIdx.x * blockDim.x + threadIdx.x;
    if (c < n) dst[(size_t)r * n + c] = gemm_out_load(src, r, c);
}

// ---- launchers --------------------------------------------------------------------------
#define BY_DTYPE(m, CALL_BF16, CALL_F32) \
    do { if ((m)->cfg.dtype == ADED_BF16) { CALL_BF16; } else { CALL_F32; } } while (0)

void launch_embed(aded_model* m, const int32_t* tokens, int rows, cudaStream_t st) {
    const int d = m->cfg.d_model;
    BY_DTYPE(m, (k_embed<bf16><<<rows, 256, 0, st>>>((const bf16*)m->top.embed, tokens, (bf16*)m->h, d, m->status)),
             (k_embed<float><<<rows, 256, 0, st>>>((const float*)m->top.embed, tokens, (float*)m->h, d, m->status)));
}

void launch_rope_table(aded_model* m, int rows, cudaStream_t st) {
    k_rope_table<<<rows, 64, 0, st>>>(m->rows.pos, m->rope_cos, m->rope_sin, m->cfg.head_dim / 2,
                                      (double)m->cfg.rope_theta, m->status);
}

void launch_add_rmsnorm(aded_model* m, const GemmOut* y, const void* gain, int rows, cudaStream_t st) {
    const int d = m->cfg.d_model;
    GemmOut none = {};
    const GemmOut& yy = y ? *y : none;
    const int has = y != nullptr;
    BY_DTYPE(m, (k_add_rmsnorm<bf16><<<rows, 256, 0, st>>>((bf16*)m->h, yy, has, (const bf16*)gain, (bf16*)m->x, d, m->cfg.rms_eps, m->status)),
             (k_add_rmsnorm<float><<<rows, 256, 0, st>>>((float*)m->h, yy, has, (const float*)gain, (float*)m->x, d, m->cfg.rms_eps, m->status)));
}

static void launch_gemm_plain(aded_model* m, const void* x, const void* w, float* y, int rows, int n, int k, cudaStream_t st) {
    dim3 grid((n + 63) / 64, (rows + 63) / 64);
    BY_DTYPE(m, (k_gemm_plain<bf16><<<grid, 256, 0, st>>>((const bf16*)x, (const bf16*)w, y, rows, n, k, m->status)),
             (k_gemm_plain<float><<<grid, 256, 0, st>>>((const float*)x, (const float*)w, y, rows, n, k, m->status)));
}

GemmOut launch_gemm(aded_model* m, int w_map, int x_map, const void* x, const void* w, float* y, int rows, int n, int k,
                    cudaStream_t st) {
    GemmOut out = {};
    out.n = n;
    out.rows = rows;
    if (m->ws_ready && w_map >= 0 && x_map >= 0 && ws_supported(n, k)) {
        // tensor-core path, 128 rows of x per pass over the weights; the result stays in slots
        for (int row0 = 0; row0 < rows; row0 += 128) {
            const int part = rows - row0 < 128 ? rows - row0 : 128;
            ws_launch(m->ws_maps[w_map], m->ws_maps[x_map], part, row0, n, k, m->ws_slots, m->status, m->device, st);
        }
        out.mode = 1;
        out.slots = m->ws_slots;
        out.n_tiles = n / 128;
        out.kb = k / 64;
        out.g = ws_grid(m->device, n, k);
        return out;
    }
    launch_gemm_plain(m, x, w, y, rows, n, k, st);
    out.mode = 0;
    out.y = y;
    return out;
}

void launch_materialize(aded_model* m, const GemmOut& src, float* dst, int rows, cudaStream_t st) {
    dim3 grid((src.n + 255) / 256, rows);
    k_materialize<<<grid, 256, 0, st>>>(src, dst, src.n, m->status);
}

void launch_rope_kv(aded_model* m, aded_kv* kv, const GemmOut& qkv, int layer, int rows, cudaStream_t st) {
    dim3 grid(rows, m->cfg.n_heads);
    const int H = m->cfg.n_heads, hd = m->cfg.head_dim;
    BY_DTYPE(m, (k_rope_kv<bf16><<<grid, 64, 0, st>>>(qkv, m->rope_cos, m->rope_sin, (bf16*)m->q, kv->base_dev, kv->cap_dev, kv->len_dev, m->rows.seq, m->rows.local, layer, H, hd, m->status)),
             (k_rope_kv<float><<<grid, 64, 0, st>>>(qkv, m->rope_cos, m->rope_sin, (float*)m->q, kv->base_dev, kv->cap_dev, kv->len_dev, m->rows.seq, m->rows.local, layer, H, hd, m->status)));
}

void launch_swiglu(aded_model* m, const GemmOut& gu, int rows, cudaStream_t st) {
    const int F = m->cfg.d_ffn;
    dim3 grid((F + 255) / 256, rows);
    BY_DTYPE(m, (k_swiglu<bf16><<<grid, 256, 0, st>>>(gu, (bf16*)m->act, F, m->status)),
             (k_swiglu<float><<<grid, 256, 0, st>>>(gu, (float*)m->act, F, m->status)));
}

void launch_argmax(aded_model* m, const GemmOut& logits, int rows, cudaStream_t st) {
    const size_t smem = logits.mode == 1 ? (size_t)logits.n_tiles * sizeof(TileRef) : 0;
    k_argmax<<<rows, 256, smem, st>>>(logits, m->best, m->cfg.vocab, m->status);
}

}  // namespace aded
