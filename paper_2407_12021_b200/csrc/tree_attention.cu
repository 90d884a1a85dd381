// Tree attention ("Draft Construction and Verification"): every tree node attends to all
// committed cache positions and, inside the tree, to its ancestors and itself only.
//
// The tree's own keys/values already sit in the cache at slots L + node index (written by the
// rotary/K-V kernel), so the key set of node i is cache[0, L) plus { L + j : bit j of anc[i] }.
//
// bf16 models: split-KV kernel on tensor cores.  A CTA owns (sequence, head, key split); each of
// its warps owns 16 tree nodes (query rows) and walks the split's keys in blocks of 64 that all
// warps share through shared memory (three-deep cp.async pipeline).  Scores S = Q K^T and O += P V
// are m16n8k16 bf16 MMAs with fp32 accumulators; the online softmax keeps a running reference and
// sum per row in registers (quad shuffles).  Numerators are 2^(t - M) with t the score in the log2
// domain and M = ceil(max t) an integer, rounded to bf16 for the P V product while the row sum keeps
// them unrounded; integer references make all rescaling exact.  Only the blocks that reach past L apply the ancestor
// bit mask.  The splits of one (sequence, head) form a thread-block cluster: each keeps its
// unnormalised partial (O, max, sum) in shared memory and the cluster combines them through
// distributed shared memory, so partials never touch global memory and no merge kernel runs.  The
// key range is derived on the device from the committed length.
//
// fp32 models use the plain one-warp-per-(row, head) kernel below.
#include "aded_internal.cuh"

namespace aded {

// ------------------------------------------------------------------------------------------
// plain kernel (fp32 models; also a readable statement of the computation)
// ------------------------------------------------------------------------------------------
template <typename T, int HD>
__global__ void __launch_bounds__(128) k_tree_attn_plain(
        const T* __restrict__ q, T* __restrict__ out, char* const* __restrict__ base,
        const int32_t* __restrict__ cap, const int32_t* __restrict__ len, const int32_t* __restrict__ row_seq,
        const uint64_t* __restrict__ anc, int layer, int H, int rows, float scale, const int32_t* status) {
    pdl_enter();
    if (first_thread_of_grid()) trace_mark(status, TK_ATTN);
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

// ------------------------------------------------------------------------------------------
// tensor-core split-KV kernel (bf16)
// ------------------------------------------------------------------------------------------
constexpr int TA_BLK = 64;   // keys per shared-memory block
constexpr int TA_STAGES = 3; // key blocks in flight per CTA (cp.async pipeline depth)

__device__ __forceinline__ void cp_async16(void* smem, const void* gmem) {
    const uint32_t s = (uint32_t)__cvta_generic_to_shared(smem);
    asm volatile("cp.async.cg.shared.global [%0], [%1], 16;" ::"r"(s), "l"(gmem) : "memory");
}
__device__ __forceinline__ void cp_async_commit() { asm volatile("cp.async.commit_group;" ::: "memory"); }
template <int N> __device__ __forceinline__ void cp_async_wait() { asm volatile("cp.async.wait_group %0;" ::"n"(N) : "memory"); }

__device__ __forceinline__ void ldmatrix_x4(uint32_t* r, const void* smem) {
    const uint32_t s = (uint32_t)__cvta_generic_to_shared(smem);
    asm volatile("ldmatrix.sync.aligned.m8n8.x4.shared.b16 {%0, %1, %2, %3}, [%4];"
                 : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]) : "r"(s));
}
__device__ __forceinline__ void ldmatrix_x4_trans(uint32_t* r, const void* smem) {
    const uint32_t s = (uint32_t)__cvta_generic_to_shared(smem);
    asm volatile("ldmatrix.sync.aligned.m8n8.x4.trans.shared.b16 {%0, %1, %2, %3}, [%4];"
                 : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]) : "r"(s));
}
__device__ __forceinline__ void mma_bf16_16816(float* c, const uint32_t* a, uint32_t b0, uint32_t b1) {
    asm volatile("mma.sync.aligned.m16n8k16.row.col.f32.bf16.bf16.f32 {%0, %1, %2, %3}, {%4, %5, %6, %7}, {%8, %9}, {%0, %1, %2, %3};"
                 : "+f"(c[0]), "+f"(c[1]), "+f"(c[2]), "+f"(c[3])
                 : "r"(a[0]), "r"(a[1]), "r"(a[2]), "r"(a[3]), "r"(b0), "r"(b1));
}
// 2^x for x <= 0 by the hardware approximation (2 ulp; results below 2^-126 flush to zero).
__device__ __forceinline__ float ex2_fast(float x) {
    float y;
    asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
    return y;
}
__device__ __forceinline__ uint32_t pack_bf16(float lo, float hi) {
    __nv_bfloat162 v = __floats2bfloat162_rn(lo, hi);
    return *reinterpret_cast<uint32_t*>(&v);
}

// Address of the 16-byte chunk `chunk` of row `row` in a [rows][HD] bf16 tile whose chunks are
// XOR-swizzled inside each group of eight (conflict-free ldmatrix over eight rows).
template <int HD>
__device__ __forceinline__ bf16* tile_chunk(bf16* tile, int row, int chunk) {
    return tile + (size_t)row * HD + (((chunk & ~7) | ((chunk ^ row) & 7)) << 3);
}

struct AttnArgs {
    const bf16* q;                 // [R][H][HD]
    bf16* out;                     // [R][H][HD] attention output
    char* const* base;
    const int32_t* cap;
    const int32_t* len;
    const int32_t* row_off;
    const uint64_t* anc;
    int layer, H, n_splits, rows_total;
    int row_blocks;                // CTAs (of NW * 16 query rows each) per sequence and key split; grid.z = batch * row_blocks
    float scale_log2;              // softmax scale * log2(e)
    const int32_t* status;
};

template <int HD, int NW>
__global__ void __launch_bounds__(NW * 32) k_tree_attn_mma(AttnArgs a) {
    pdl_launch_dependents();
    constexpr int CHUNKS = HD / 8;         // 16-byte chunks per row
    extern __shared__ __align__(128) uint8_t smem_raw[];
    bf16* sk = reinterpret_cast<bf16*>(smem_raw);                 // [TA_STAGES][TA_BLK][HD]
    bf16* sv = sk + TA_STAGES * TA_BLK * HD;                      // [TA_STAGES][TA_BLK][HD]
    // Before waiting for the previous kernel (which writes the tree's own K/V rows and q): start
    // fetching this CTA's first key blocks if they lie entirely in the committed part of the cache,
    // which no kernel of this pass writes.  The committed length and the tree size were written before
    // this pass began (a pass opens with a copy on the stream, which no kernel of the pass overtakes),
    // but this kernel does not rely on that: both are read again after the wait and the early blocks
    // are used only if the two reads agree, otherwise they are fetched again.
    // The cache block's address and capacity never change after the cache was created.
    const int pre_hh = blockIdx.x, pre_b = blockIdx.z / a.row_blocks;
    const size_t pre_cp = a.cap[pre_b];
    const bf16* pre_kg = reinterpret_cast<const bf16*>(a.base[pre_b]) + (((size_t)a.layer * 2 + 0) * a.H + pre_hh) * pre_cp * HD;
    const bf16* pre_vg = reinterpret_cast<const bf16*>(a.base[pre_b]) + (((size_t)a.layer * 2 + 1) * a.H + pre_hh) * pre_cp * HD;
    __shared__ int s_pre[2];               // one thread reads, so that the whole CTA acts on the same values
    if (threadIdx.x == 0) {
        s_pre[0] = __ldcg(a.len + pre_b);
        s_pre[1] = __ldcg(a.row_off + pre_b + 1) - __ldcg(a.row_off + pre_b);
    }
    __syncthreads();
    const int pre_L = s_pre[0], pre_T = s_pre[1];
    int pre_blk0 = 0, n_pre = 0;
    if (pre_L >= 0 && pre_T >= 1 && pre_T <= ADED_MAX_NODES && (size_t)pre_L + pre_T <= pre_cp) {
        const int nb_p = (pre_L + pre_T + TA_BLK - 1) / TA_BLK;
        const int bps_p = (nb_p + a.n_splits - 1) / a.n_splits;
        pre_blk0 = blockIdx.y * bps_p;
        const int blk1_p = min(nb_p, pre_blk0 + bps_p);
#pragma unroll
        for (int st = 0; st < TA_STAGES - 1; ++st) {
            const int blk = pre_blk0 + st;
            if (n_pre == st && blk < blk1_p && (blk + 1) * TA_BLK <= pre_L) {
                bf16* dk = sk + (size_t)st * TA_BLK * HD;
                bf16* dv = sv + (size_t)st * TA_BLK * HD;
                for (int e = threadIdx.x; e < TA_BLK * CHUNKS; e += NW * 32) {
                    const int row = e / CHUNKS, chunk = e % CHUNKS;
                    const size_t pos = (size_t)blk * TA_BLK + row;
                    cp_async16(tile_chunk<HD>(dk, row, chunk), pre_kg + pos * HD + chunk * 8);
                    cp_async16(tile_chunk<HD>(dv, row, chunk), pre_vg + pos * HD + chunk * 8);
                }
                cp_async_commit();
                ++n_pre;
            }
        }
    }
    pdl_wait();
    if (first_thread_of_grid()) trace_mark(a.status, TK_ATTN);
    // The status word is fetched along with the rest of the call's metadata and acted on before the
    // first store, so that it does not cost a memory round trip of its own.  Until then nothing is
    // written, and every load below stays inside the cache block and the row arrays whatever a failed
    // earlier kernel left in them (positions are clamped to the capacity).
    const int pass_status = *a.status;
    constexpr int KSTEPS = HD / 16;        // k steps of Q K^T
    constexpr int ONT = HD / 8;            // n tiles of the output

    const int hh = blockIdx.x, split = blockIdx.y, b = blockIdx.z / a.row_blocks;
    const int row_base = (blockIdx.z % a.row_blocks) * NW * 16;    // first query row (node of the tree) of this CTA
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31, g = lane >> 2, tig = lane & 3;
    const int off = a.row_off[b];
    const int T = a.row_off[b + 1] - off;
    const int L = __ldcg(a.len + b);
    const size_t cp = a.cap[b];
    const int n_keys = L + T;
    const int nb = (n_keys + TA_BLK - 1) / TA_BLK;
    const int bps = (nb + a.n_splits - 1) / a.n_splits;
    const int blk0 = split * bps;
    const int blk1 = min(nb, blk0 + bps);

    // this thread's two query rows (local node indices) and their global rows
    const int i0 = row_base + warp * 16 + g, i1 = i0 + 8;
    const bool v0 = i0 < T, v1 = i1 < T;
    const bf16* kg = reinterpret_cast<const bf16*>(a.base[b]) + (((size_t)a.layer * 2 + 0) * a.H + hh) * cp * HD;
    const bf16* vg = reinterpret_cast<const bf16*>(a.base[b]) + (((size_t)a.layer * 2 + 1) * a.H + hh) * cp * HD;

    // Q fragments straight from global memory in the MMA A layout
    uint32_t qf[KSTEPS][4];
    {
        const bf16* q0 = a.q + ((size_t)(off + (v0 ? i0 : 0)) * a.H + hh) * HD;
        const bf16* q1 = a.q + ((size_t)(off + (v1 ? i1 : 0)) * a.H + hh) * HD;
#pragma unroll
        for (int ks = 0; ks < KSTEPS; ++ks) {
            const int c = ks * 16 + 2 * tig;
            qf[ks][0] = v0 ? *reinterpret_cast<const uint32_t*>(q0 + c) : 0u;
            qf[ks][1] = v1 ? *reinterpret_cast<const uint32_t*>(q1 + c) : 0u;
            qf[ks][2] = v0 ? *reinterpret_cast<const uint32_t*>(q0 + c + 8) : 0u;
            qf[ks][3] = v1 ? *reinterpret_cast<const uint32_t*>(q1 + c + 8) : 0u;
        }
    }
    uint64_t m0lo = 0, m0hi = 0, m1lo = 0, m1hi = 0;             // ancestor bit sets of the two rows
    if (v0) { m0lo = a.anc[2 * (off + i0)]; m0hi = a.anc[2 * (off + i0) + 1]; }
    if (v1) { m1lo = a.anc[2 * (off + i1)]; m1hi = a.anc[2 * (off + i1) + 1]; }

    float oacc[ONT][4];
#pragma unroll
    for (int n = 0; n < ONT; ++n) { oacc[n][0] = oacc[n][1] = oacc[n][2] = oacc[n][3] = 0.f; }
    float mrow0 = -INFINITY, mrow1 = -INFINITY, lrow0 = 0.f, lrow1 = 0.f;

    auto load_block = [&](int blk, int buf) {
        // positions past the last key are clamped to it (they are masked below); the clamp keeps
        // every address inside the rows this call may touch
        const int p0 = blk * TA_BLK;
        bf16* dk = sk + (size_t)buf * TA_BLK * HD;
        bf16* dv = sv + (size_t)buf * TA_BLK * HD;
        for (int e = threadIdx.x; e < TA_BLK * CHUNKS; e += NW * 32) {
            const int row = e / CHUNKS, chunk = e % CHUNKS;
            const int pos = min(min(p0 + row, n_keys - 1), (int)cp - 1);
            cp_async16(tile_chunk<HD>(dk, row, chunk), kg + (size_t)pos * HD + chunk * 8);
            cp_async16(tile_chunk<HD>(dv, row, chunk), vg + (size_t)pos * HD + chunk * 8);
        }
        cp_async_commit();
    };

    // Pipeline: TA_STAGES - 1 blocks are in flight while one is being used.  Every iteration commits
    // exactly one group (an empty one past the end), so "all but the newest TA_STAGES - 2 groups have
    // landed" always means the current block has.  (A split past the last key block has nothing to do
    // but still joins the merge.)
    if (n_pre > 0 && (L != pre_L || T != pre_T || blk0 != pre_blk0)) {
        // the early reads were stale: let the early copies land, then fetch the right blocks over them
        cp_async_wait<0>();
        __syncthreads();
        n_pre = 0;
    }
#pragma unroll
    for (int s = 0; s < TA_STAGES - 1; ++s) {
        if (s < n_pre) continue;           // already in flight
        if (blk0 + s < blk1) load_block(blk0 + s, s); else cp_async_commit();
    }
    for (int blk = blk0; blk < blk1; ++blk) {
        const int buf = (blk - blk0) % TA_STAGES;
        cp_async_wait<TA_STAGES - 2>();
        __syncthreads();                      // block `blk` is visible; everyone is done with block blk - 1
        {
            const int nxt = blk + TA_STAGES - 1;   // goes into the buffer block blk - 1 used
            if (nxt < blk1) load_block(nxt, (nxt - blk0) % TA_STAGES); else cp_async_commit();
        }
        bf16* tk = sk + (size_t)buf * TA_BLK * HD;
        bf16* tv = sv + (size_t)buf * TA_BLK * HD;

        // ---- S = Q K^T for 64 keys: 8 n tiles x KSTEPS k steps ----
        float sacc[TA_BLK / 8][4];
#pragma unroll
        for (int n = 0; n < TA_BLK / 8; ++n) { sacc[n][0] = sacc[n][1] = sacc[n][2] = sacc[n][3] = 0.f; }
#pragma unroll
        for (int ks = 0; ks < KSTEPS; ++ks) {
#pragma unroll
            for (int np = 0; np < TA_BLK / 16; ++np) {
                uint32_t kb[4];
                const int row = np * 16 + (lane & 7) + ((lane >> 4) << 3);
                const int chunk = ks * 2 + ((lane >> 3) & 1);
                ldmatrix_x4(kb, tile_chunk<HD>(tk, row, chunk));
                mma_bf16_16816(sacc[2 * np], qf[ks], kb[0], kb[1]);
                mma_bf16_16816(sacc[2 * np + 1], qf[ks], kb[2], kb[3]);
            }
        }
        // ---- scale, mask, online softmax ----
        const int p0 = blk * TA_BLK;
        const bool need_mask = p0 + TA_BLK > L;
        float bm0 = -INFINITY, bm1 = -INFINITY;
#pragma unroll
        for (int n = 0; n < TA_BLK / 8; ++n) {
#pragma unroll
            for (int e = 0; e < 4; ++e) {
                float s = sacc[n][e];          // raw dot product; the scale (> 0) is applied to the maximum and inside the exponent
                if (need_mask) {
                    const int pos = p0 + n * 8 + 2 * tig + (e & 1);
                    const int j = pos - L;
                    bool ok = j < 0;
                    if (!ok && j < T) {
                        const uint64_t lo = e < 2 ? m0lo : m1lo, hi = e < 2 ? m0hi : m1hi;
                        ok = j < 64 ? (lo >> j) & 1 : (hi >> (j - 64)) & 1;
                    }
                    if (!ok) s = -INFINITY;
                }
                sacc[n][e] = s;
                if (e < 2) bm0 = fmaxf(bm0, s); else bm1 = fmaxf(bm1, s);
            }
        }
        bm0 = fmaxf(bm0, __shfl_xor_sync(0xffffffffu, bm0, 1));
        bm0 = fmaxf(bm0, __shfl_xor_sync(0xffffffffu, bm0, 2));
        bm1 = fmaxf(bm1, __shfl_xor_sync(0xffffffffu, bm1, 1));
        bm1 = fmaxf(bm1, __shfl_xor_sync(0xffffffffu, bm1, 2));
        // The running reference is the maximum rounded UP to an integer (scores are in the log2
        // domain), so every rescale below is an exact power of two and the bf16 rounding of the
        // numerators 2^(t - M) does not depend on how the keys are split or ordered.
        const float nm0 = fmaxf(mrow0, ceilf(bm0 * a.scale_log2)), nm1 = fmaxf(mrow1, ceilf(bm1 * a.scale_log2));
        const float use0 = nm0 == -INFINITY ? 0.f : nm0, use1 = nm1 == -INFINITY ? 0.f : nm1;
        // the partial sums need rescaling only when a row's reference moved (rare after the first block:
        // it is an integer); a row without any key yet holds zeros, which need none
        const bool moved = (mrow0 != nm0 && mrow0 != -INFINITY) || (mrow1 != nm1 && mrow1 != -INFINITY);
        const float corr0 = exp2f(mrow0 - use0), corr1 = exp2f(mrow1 - use1);
        mrow0 = nm0;
        mrow1 = nm1;
        float ps0 = 0.f, ps1 = 0.f;
        uint32_t pf[TA_BLK / 16][4];
#pragma unroll
        for (int n = 0; n < TA_BLK / 8; ++n) {
            const float e0 = ex2_fast(fmaf(sacc[n][0], a.scale_log2, -use0)), e1 = ex2_fast(fmaf(sacc[n][1], a.scale_log2, -use0));
            const float e2 = ex2_fast(fmaf(sacc[n][2], a.scale_log2, -use1)), e3 = ex2_fast(fmaf(sacc[n][3], a.scale_log2, -use1));
            ps0 += e0 + e1;
            ps1 += e2 + e3;
            pf[n >> 1][(n & 1) * 2 + 0] = pack_bf16(e0, e1);
            pf[n >> 1][(n & 1) * 2 + 1] = pack_bf16(e2, e3);
        }
        if (__any_sync(0xffffffffu, moved)) {
            lrow0 *= corr0;
            lrow1 *= corr1;
#pragma unroll
            for (int n = 0; n < ONT; ++n) {
                oacc[n][0] *= corr0; oacc[n][1] *= corr0;
                oacc[n][2] *= corr1; oacc[n][3] *= corr1;
            }
        }
        lrow0 += ps0;
        lrow1 += ps1;
        // ---- O += P V ----
#pragma unroll
        for (int kk = 0; kk < TA_BLK / 16; ++kk) {
#pragma unroll
            for (int np = 0; np < ONT / 2; ++np) {
                uint32_t vb[4];
                const int row = kk * 16 + (lane & 7) + (((lane >> 3) & 1) << 3);
                const int chunk = np * 2 + (lane >> 4);
                ldmatrix_x4_trans(vb, tile_chunk<HD>(tv, row, chunk));
                mma_bf16_16816(oacc[2 * np], pf[kk], vb[0], vb[1]);
                mma_bf16_16816(oacc[2 * np + 1], pf[kk], vb[2], vb[3]);
            }
        }
    }
    // ---- merge the splits of this (sequence, head) across the cluster ----
    // Every CTA parks its unnormalised partial (O, running max, sum) in its own shared memory; after a
    // cluster barrier CTA j combines rows j, j + S, ... from all S CTAs' shared memory (distributed
    // shared memory reads), out = sum_s O_s 2^(m_s - M) / sum_s l_s 2^(m_s - M), rounds to bf16 and
    // writes the attention output.  No partial ever goes to global memory.
    if (pass_status != 0) return;     // uniform over the cluster: nobody waits for a CTA that left
    lrow0 += __shfl_xor_sync(0xffffffffu, lrow0, 1);
    lrow0 += __shfl_xor_sync(0xffffffffu, lrow0, 2);
    lrow1 += __shfl_xor_sync(0xffffffffu, lrow1, 1);
    lrow1 += __shfl_xor_sync(0xffffffffu, lrow1, 2);
    __syncthreads();                                   // all warps are done with the K/V tiles
    float* so = reinterpret_cast<float*>(smem_raw);    // [NW*16][HD]
    float* sml = so + NW * 16 * HD;                    // [NW*16][2]
    {
        const int r0 = warp * 16 + g, r1 = r0 + 8;
#pragma unroll
        for (int n = 0; n < ONT; ++n) {
            *reinterpret_cast<float2*>(so + (size_t)r0 * HD + n * 8 + 2 * tig) = make_float2(oacc[n][0], oacc[n][1]);
            *reinterpret_cast<float2*>(so + (size_t)r1 * HD + n * 8 + 2 * tig) = make_float2(oacc[n][2], oacc[n][3]);
        }
        if (tig == 0) {
            sml[r0 * 2] = mrow0; sml[r0 * 2 + 1] = lrow0;
            sml[r1 * 2] = mrow1; sml[r1 * 2 + 1] = lrow1;
        }
    }
    const int S = a.n_splits;
    if (S > 1) {
        asm volatile("barrier.cluster.arrive.release.aligned;" ::: "memory");
        asm volatile("barrier.cluster.wait.acquire.aligned;" ::: "memory");
    } else {
        __syncthreads();
    }
    const uint32_t so_addr = (uint32_t)__cvta_generic_to_shared(so), sml_addr = (uint32_t)__cvta_generic_to_shared(sml);
    constexpr int QUADS = HD / 4;                      // float4 groups per row
    const int t_here = min(max(T - row_base, 0), NW * 16);         // query rows of this CTA
    for (int item = threadIdx.x; item < ((t_here - split + S - 1) / S) * QUADS; item += NW * 32) {
        const int row = split + (item / QUADS) * S, c4 = (item % QUADS) * 4;       // row inside this CTA's block
        // all remote reads of an item are issued before any is used (S <= 8 partials)
        float ms[8], ls[8];
        float4 os[8];
        float M = -INFINITY;
#pragma unroll
        for (int s2 = 0; s2 < 8; ++s2) {
            ms[s2] = -INFINITY;
            ls[s2] = 0.f;
            os[s2] = make_float4(0.f, 0.f, 0.f, 0.f);
            if (s2 < S) {
                uint32_t rm, ro;
                asm volatile("mapa.shared::cluster.u32 %0, %1, %2;" : "=r"(rm) : "r"(sml_addr + (uint32_t)row * 8), "r"(s2));
                asm volatile("mapa.shared::cluster.u32 %0, %1, %2;" : "=r"(ro) : "r"(so_addr + (uint32_t)(row * HD + c4) * 4), "r"(s2));
                asm volatile("ld.shared::cluster.v2.f32 {%0, %1}, [%2];" : "=f"(ms[s2]), "=f"(ls[s2]) : "r"(rm));
                asm volatile("ld.shared::cluster.v4.f32 {%0, %1, %2, %3}, [%4];"
                             : "=f"(os[s2].x), "=f"(os[s2].y), "=f"(os[s2].z), "=f"(os[s2].w) : "r"(ro));
            }
        }
#pragma unroll
        for (int s2 = 0; s2 < 8; ++s2) M = fmaxf(M, ms[s2]);
        float4 num = make_float4(0.f, 0.f, 0.f, 0.f);
        float den = 0.f;
#pragma unroll
        for (int s2 = 0; s2 < 8; ++s2) {
            if (ms[s2] == -INFINITY) continue;     // an empty split (or s2 >= S) holds no keys of this row
            const float w = exp2f(ms[s2] - M);
            den += ls[s2] * w;
            num.x += os[s2].x * w; num.y += os[s2].y * w; num.z += os[s2].z * w; num.w += os[s2].w * w;
        }
        const float inv = 1.f / den;
        bf16* dst = a.out + ((size_t)(off + row_base + row) * a.H + hh) * HD + c4;
        const __nv_bfloat162 lo = __floats2bfloat162_rn(num.x * inv, num.y * inv), hi = __floats2bfloat162_rn(num.z * inv, num.w * inv);
        uint2 u;
        u.x = *reinterpret_cast<const uint32_t*>(&lo);
        u.y = *reinterpret_cast<const uint32_t*>(&hi);
        *reinterpret_cast<uint2*>(dst) = u;
    }
    if (S > 1) {   // nobody may leave while a neighbour still reads its shared memory
        asm volatile("barrier.cluster.arrive.release.aligned;" ::: "memory");
        asm volatile("barrier.cluster.wait.acquire.aligned;" ::: "memory");
    }
}

template <int HD, int NW>
static size_t attn_smem() {
    const size_t kv = (size_t)2 * TA_STAGES * TA_BLK * HD * sizeof(bf16), merge = (size_t)NW * 16 * (HD + 2) * sizeof(float);
    return kv > merge ? kv : merge;
}

template <int HD, int NW>
static void launch_mma_nw(aded_model* m, AttnArgs& a, int batch, int splits, cudaStream_t st) {
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3(m->cfg.n_heads, splits, batch * a.row_blocks);
    cfg.blockDim = dim3(NW * 32);
    cfg.dynamicSmemBytes = attn_smem<HD, NW>();
    cfg.stream = st;
    cudaLaunchAttribute attr[2];
    int n = 0;
    if (splits > 1) {
        attr[n].id = cudaLaunchAttributeClusterDimension;
        attr[n].val.clusterDim.x = 1;
        attr[n].val.clusterDim.y = splits;
        attr[n].val.clusterDim.z = 1;
        ++n;
    }
    attr[n].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[n].val.programmaticStreamSerializationAllowed = 1;
    ++n;
    cfg.attrs = attr;
    cfg.numAttrs = n;
    cudaLaunchKernelEx(&cfg, k_tree_attn_mma<HD, NW>, a);
}

template <int HD>
static void launch_mma(aded_model* m, aded_kv* kv, int layer, int batch, int rows, int max_tree, cudaStream_t st) {
    AttnArgs a;
    a.q = (const bf16*)m->q;
    a.out = (bf16*)m->attn;
    a.base = kv->base_dev;
    a.cap = kv->cap_dev;
    a.len = kv->len_dev;
    a.row_off = m->seqs.row_off;
    a.anc = m->rows.anc;
    a.layer = layer;
    a.H = m->cfg.n_heads;
    // Trees of more than 64 nodes are worked as two blocks of 64 query rows by separate CTAs (four
    // warps and two CTAs per SM as for small trees; an eight-warp CTA holds a whole SM's registers and
    // left the launch at one CTA per SM in two waves).  Key splits per (sequence, head, row block): up
    // to 8 (one thread-block cluster), as many as keep the launch within the two-per-SM CTA slots.
    a.row_blocks = max_tree <= 64 ? 1 : 2;
    int splits = ws_grid_limit(m->device) / (m->cfg.n_heads * batch * a.row_blocks);
    splits = splits < 1 ? 1 : splits > 8 ? 8 : splits;
    a.n_splits = splits;
    a.rows_total = rows;
    a.scale_log2 = 1.4426950408889634f / sqrtf((float)HD);
    a.status = m->status;
    launch_mma_nw<HD, 4>(m, a, batch, splits, st);
}

// Raises the split-KV kernels' dynamic shared-memory limit; once per process, before any launch.
bool attn_prepare() {
    bool ok = true;
    ok &= cudaFuncSetAttribute(k_tree_attn_mma<128, 4>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)attn_smem<128, 4>()) == cudaSuccess;
    ok &= cudaFuncSetAttribute(k_tree_attn_mma<64, 4>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)attn_smem<64, 4>()) == cudaSuccess;
    return ok;
}

void launch_tree_attention(aded_model* m, aded_kv* kv, int layer, int batch, int rows, int max_tree, cudaStream_t st) {
    const int H = m->cfg.n_heads, hd = m->cfg.head_dim;
    if (m->att_tc && kv->maps_dev) {
        launch_tree_attention_tc(m, kv, layer, batch, max_tree, st);
        return;
    }
    if (m->cfg.dtype == ADED_BF16 && m->att_mma) {
        if (hd == 128) launch_mma<128>(m, kv, layer, batch, rows, max_tree, st);
        else launch_mma<64>(m, kv, layer, batch, rows, max_tree, st);
        return;
    }
    const float scale = 1.f / sqrtf((float)hd);
    const int warps = rows * H;
    const int blocks = (warps + 3) / 4;
#define ATTN(T, HD)                                                                                          \
    launch_k(k_tree_attn_plain<T, HD>, blocks, 128, 0, st, (const T*)m->q, (T*)m->attn, kv->base_dev, kv->cap_dev, \
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
