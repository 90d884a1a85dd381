// Tree attention ("Draft Construction and Verification"): every tree node attends to all
// committed cache positions and, inside the tree, to its ancestors and itself only.
//
// The tree's own keys/values already sit in the cache at slots L + node index (written by the
// rotary/K-V kernel), so the key set of node i is cache[0, L) plus { L + j : bit j of anc[i] }.
#include "aded_internal.cuh"

namespace aded {

// Plain version: one warp per (row, head).  The lanes split head_dim; each key costs a warp
// reduction for the score and one online-softmax update (running max m, running sum l, and
// hd/32 output elements per lane).  Scores and probabilities are fp32 throughout.
template <typename T, int HD>
__global__ void __launch_bounds__(128) k_tree_attn_plain(
        const T* __restrict__ q, T* __restrict__ out, char* const* __restrict__ base,
        const int32_t* __restrict__ cap, const int32_t* __restrict__ len, const int32_t* __restrict__ row_seq,
        const uint64_t* __restrict__ anc, int layer, int H, int rows, float scale, const int32_t* status) {
    if (*status != 0) return;
    constexpr int PER = HD / 32;
    const int warp = blockIdx.x * (blockDim.x >> 5) + (threadIdx.x >> 5);
    const int lane = threadIdx.x & 31;
    if (warp >= rows * H) return;
    const int r = warp / H, hh = warp % H;
    const int b = row_seq[r];
    const int L = len[b];
    const size_t cp = cap[b];
    const T* kbase = reinterpret_cast<const T*>(base[b]) + (((size_t)layer * 2 + 0) * H + hh) * cp * HD;
    const T* vbase = reinterpret_cast<const T*>(base[b]) + (((size_t)layer * 2 + 1) * H + hh) * cp * HD;
    float qv[PER], acc[PER];
#pragma unroll
    for (int e = 0; e < PER; ++e) {
        qv[e] = to_f32(q[((size_t)r * H + hh) * HD + lane * PER + e]);
        acc[e] = 0.f;
    }
    float mx = -INFINITY, sum = 0.f;
    const uint64_t a_lo = anc[2 * r], a_hi = anc[2 * r + 1];
    const int n_keys = L + ADED_MAX_NODES;
    for (int p = 0; p < n_keys; ++p) {
        if (p >= L) {
            const int j = p - L;
            const bool on = j < 64 ? (a_lo >> j) & 1 : (a_hi >> (j - 64)) & 1;
            if (!on) continue;
        }
        const T* kr = kbase + (size_t)p * HD + lane * PER;
        float s = 0.f;
#pragma unroll
        for (int e = 0; e < PER; ++e) s = fmaf(qv[e], to_f32(kr[e]), s);
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) s += __shfl_xor_sync(0xffffffffu, s, o);
        s *= scale;
        const float nm = fmaxf(mx, s);
        const float corr = expf(mx - nm), pr = expf(s - nm);
        sum = sum * corr + pr;
        const T* vr = vbase + (size_t)p * HD + lane * PER;
#pragma unroll
        for (int e = 0; e < PER; ++e) acc[e] = fmaf(pr, to_f32(vr[e]), acc[e] * corr);
        mx = nm;
    }
    const float inv = 1.f / sum;
#pragma unroll
    for (int e = 0; e < PER; ++e) out[((size_t)r * H + hh) * HD + lane * PER + e] = from_f32<T>(acc[e] * inv);
}

void launch_tree_attention(aded_model* m, aded_kv* kv, int layer, int batch, int rows, cudaStream_t st) {
    (void)batch;
    const int H = m->cfg.n_heads, hd = m->cfg.head_dim;
    const float scale = 1.f / sqrtf((float)hd);
    const int warps = rows * H;
    const int blocks = (warps + 3) / 4;
#define ATTN(T, HD)                                                                                          \
    k_tree_attn_plain<T, HD><<<blocks, 128, 0, st>>>((const T*)m->q, (T*)m->attn, kv->base_dev, kv->cap_dev, \
                                                     kv->len_dev, m->rows.seq, m->rows.anc, layer, H, rows,  \
                                                     scale, m->status)
    if (m->cfg.dtype == ADED_BF16) {
        if (hd == 128) ATTN(bf16, 128); else ATTN(bf16, 64);
    } else {
        if (hd == 128) ATTN(float, 128); else ATTN(float, 64);
    }
#undef ATTN
}

}  // namespace aded
