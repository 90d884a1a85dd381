// Weight-streaming bf16 GEMM for the decoder's projections, FFN and LM head on the 5th-generation
// tensor cores (tcgen05, accumulators in TMEM, operands staged by TMA); the LM head's variant also
// reduces its result to per-tile greedy candidates in the kernel's tail.
//
//   y[r, n] = sum_k x[r, k] * w[n, k]        r < rows <= 256,  w row-major [N, K], x row-major [R, K]
//
// A verification step multiplies at most 128 tree nodes with every weight matrix, so the kernel is
// bound by reading W once from HBM.  Mapping:
//   * the 128 rows of a W tile are the M dimension of the MMA (all 128 TMEM lanes busy), the tree
//     nodes are its N dimension (rows padded to a multiple of 16), K advances 64 elements (one
//     128-byte swizzled line) per pipeline stage;
//   * work = (W tile, k block) units, split evenly over all resident CTAs (two per SM), so every CTA
//     streams the same number of bytes whatever N and K are; a CTA's range covers the tail of one
//     tile, whole tiles, and the head of another;
//   * a CTA stores the fp32 partial tile of each of its segments to a slot (gemm_out.cuh); the kernel
//     that consumes the result (rotary/K-V write, residual add + RMSNorm, SwiGLU) adds a tile's slots
//     in CTA order -- a fixed order, so results do not depend on timing -- and the GEMM itself ends
//     without counters, fences or dependent reads.  The consumers are small kernels of their own on
//     purpose: while one runs, the next projection's CTAs are already resident and stream their
//     first W tiles.  (Measured on a 32-layer step: folding the consumers into this kernel's tail,
//     the contributors of a tile meeting at a counter, made every projection 7-9 us longer for a
//     consumer kernel of 4-8 us saved, because the next projection then starts cold.)
//   * the LM head alone has such a tail (template parameter): the CTAs that contributed to a tile meet
//     at a counter in global memory and each reduces a share of the tile's rows to per-row greedy
//     candidates (best logit of the tile's 128 columns), so the [rows, vocab] logits are never
//     gathered by a later kernel.  All CTAs of a launch are resident at once (at most two per SM
//     are launched), so the meeting cannot deadlock; the wait is bounded all the same.  The counters
//     are never reset: launch number e waits for n x e arrivals (arithmetic modulo 2^32);
//   * the kernel is launched with programmatic dependent launch: its blocks become resident while
//     the previous kernel drains, set up barriers and TMEM, and already stream their first W tiles;
//     only the loads of x wait for the previous kernel;
//   * warp 0 issues TMA loads, warp 1 issues MMAs, warps 2..5 drain TMEM; two TMEM accumulators let
//     the MMAs of the next segment run under the drain of the last; all six warps run the LM head's tail.
// Every wait is bounded; a wait that runs out raises ADED_ERR_TIMEOUT in the status word and the
// CTA unwinds (drains its own copies, frees TMEM).
#include <cuda.h>

#include <cstdio>

#include "aded_internal.cuh"
#include "gemm_out.cuh"
#include "tc_ptx.cuh"

namespace aded {

constexpr int WS_BM = 128;           // W rows per tile (MMA M)
constexpr int WS_BK = 64;            // k elements per stage (128 bytes of bf16)
constexpr int WS_THREADS = 192;
constexpr long long WS_MEET_CYCLES = 400000000ll;   // about 0.2 s of SM clock: limit of the wait at a counter
constexpr int WS_GMAX = 16;          // tile groups of a CTA handled per round of its tail

struct WsParams {
    int rows;            // valid rows of x
    int rb;              // rows padded to a multiple of 16 = MMA N
    int row0;            // first row of x / y handled by this launch
    int n, k;            // W is [n, k]
    int n_tiles, kb;     // tiles of 128 W rows, k blocks per tile
    int stages;
    int tmem_cols;       // power of two >= n_acc * rb
    int n_acc;           // TMEM accumulators: two (the next segment's MMAs run under the drain) up to 128 rows, one beyond
    int trace_kind;
    int narrow;          // units * (CTAs + 1) < 2^31: the work split can be computed in 32-bit arithmetic
    float* slots;        // this row block's slot region: [n_tiles + gridDim.x][rb][128] fp32
    const uint8_t* w_tiled;  // W re-tiled (ws_retile): unit (tile, k block) is 16 KB at (tile * kb + k block) * 16 KB, swizzled as staged
    int32_t* status;
    WsEpilogue epi;
};

// One contiguous copy of `bytes` (a multiple of 16, both addresses 16-byte aligned) from global to shared memory,
// completing on an mbarrier like a tensor-map copy.
__device__ __forceinline__ void bulk_load_hint(void* dst, const void* src, uint32_t bytes, uint64_t* bar, uint64_t policy) {
    asm volatile(
        "cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes.L2::cache_hint [%0], [%1], %2, [%3], %4;"
        ::"r"(smem_u32(dst)), "l"(src), "r"(bytes), "r"(smem_u32(bar)), "l"(policy) : "memory");
}

// Waits until the counter has reached `target` (arrivals are counted modulo 2^32 and never reset).
__device__ __forceinline__ bool ws_poll(const uint32_t* counter, uint32_t target, long long limit = WS_MEET_CYCLES) {
    const long long t0 = clock64();
    for (uint32_t spin = 0;; ++spin) {
        uint32_t v;
        asm volatile("ld.acquire.gpu.global.u32 %0, [%1];" : "=r"(v) : "l"(counter) : "memory");
        if ((int32_t)(v - target) >= 0) return true;
        if ((spin & 63) == 63 && clock64() - t0 > limit) return false;
    }
}
__device__ __forceinline__ void ws_arrive(uint32_t* counter) {
    asm volatile("red.release.gpu.global.add.u32 [%0], 1;" ::"l"(counter) : "memory");
}
// ws_owner (gemm_out.cuh) in 32-bit arithmetic when the products fit.
__device__ __forceinline__ int ws_owner_dev(long long u, long long units, long long G, bool narrow) {
    if (!narrow) return ws_owner(u, units, G);
    const int u32 = (int)u, n32 = (int)units, g32 = (int)G;
    int c = ((u32 + 1) * g32 - 1) / n32;
    if (c >= g32) c = g32 - 1;
    while (c > 0 && c * n32 / g32 > u32) --c;
    while (c + 1 < g32 && (c + 1) * n32 / g32 <= u32) ++c;
    return c;
}

// Sum of a tile's slots (CTA order) for four adjacent columns of local row r.
__device__ __forceinline__ float4 ws_sum4(const float* slots, const TileRef& t, int rb, int r, int col) {
    const float* p = slots + ((size_t)t.first_slot * rb + r) * WS_BM + col;
    const size_t stride = (size_t)rb * WS_BM;
    float4 sum = make_float4(0.f, 0.f, 0.f, 0.f);
    constexpr int B = 12;
    for (int i0 = 0; i0 < t.count; i0 += B) {
        float4 v[B];
#pragma unroll
        for (int j = 0; j < B; ++j)
            v[j] = i0 + j < t.count ? __ldcg(reinterpret_cast<const float4*>(p + (size_t)(i0 + j) * stride)) : make_float4(0.f, 0.f, 0.f, 0.f);
#pragma unroll
        for (int j = 0; j < B; ++j)
            if (i0 + j < t.count) sum = f4_add(sum, v[j]);
    }
    return sum;
}

// LM head: a warp per row; the best (value, lowest column) of the tile's 128 logits goes to
// cand_val / cand_idx [row][tile].
__device__ __forceinline__ void ws_row_argmax(const WsParams& p, const TileRef& t, int vt, int r, int lane, bool store) {
    const float4 v = ws_sum4(p.slots, t, p.rb, r, lane * 4);
    float bv = v.x;
    int bi = vt * WS_BM + lane * 4;
    if (v.y > bv) { bv = v.y; bi = vt * WS_BM + lane * 4 + 1; }
    if (v.z > bv) { bv = v.z; bi = vt * WS_BM + lane * 4 + 2; }
    if (v.w > bv) { bv = v.w; bi = vt * WS_BM + lane * 4 + 3; }
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) {
        const float ov = __shfl_xor_sync(0xffffffffu, bv, o);
        const int oi = __shfl_xor_sync(0xffffffffu, bi, o);
        if (ov > bv || (ov == bv && oi < bi)) { bv = ov; bi = oi; }
    }
    if (lane == 0 && store) {
        p.epi.cand_val[(size_t)(p.row0 + r) * p.n_tiles + vt] = bv;
        p.epi.cand_idx[(size_t)(p.row0 + r) * p.n_tiles + vt] = bi;
    }
}

template <bool TAIL>
__global__ void __launch_bounds__(WS_THREADS, 2)
k_gemm_ws(const __grid_constant__ CUtensorMap map_w, const __grid_constant__ CUtensorMap map_x, const __grid_constant__ CUtensorMap map_x64,
          const __grid_constant__ WsParams p) {
    extern __shared__ __align__(1024) uint8_t smem_raw[];
    // carve: stages x (W tile 16 KB | x tile rb*128 B), then barriers
    uint8_t* base = (uint8_t*)(((uintptr_t)smem_raw + 1023) & ~(uintptr_t)1023);
    const uint32_t a_bytes = WS_BM * 128, b_bytes = (uint32_t)p.rb * 128, stage_bytes = a_bytes + b_bytes;
    uint64_t* bars = (uint64_t*)(base + (size_t)p.stages * stage_bytes);
    uint64_t* full = bars;
    uint64_t* empty = bars + p.stages;
    uint64_t* acc_full = bars + 2 * p.stages;
    uint64_t* acc_empty = acc_full + 2;
    uint32_t* s_tmem = (uint32_t*)(acc_empty + 2);
    volatile int* s_flag = (volatile int*)(s_tmem + 1);   // [0] abort, [2] live, [3] meeting result

    pdl_launch_dependents();   // the next kernel may start its preamble; it waits for this one's results itself
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const long long units = (long long)p.n_tiles * p.kb;
    const long long G = gridDim.x;
    const long long u0 = ws_start(blockIdx.x, units, G), u1 = ws_start(blockIdx.x + 1, units, G);

    if (threadIdx.x == 0) {
        for (int s = 0; s < p.stages; ++s) { mbar_init(&full[s], 1); mbar_init(&empty[s], 1); }
        for (int a = 0; a < 2; ++a) { mbar_init(&acc_full[a], 1); mbar_init(&acc_empty[a], 4); }
        s_flag[0] = 0;
        s_flag[1] = 0;
        s_flag[2] = *p.status == 0;
        s_flag[3] = 1;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
        asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
    }
    if (warp == 1) {
        asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(s_tmem)), "r"((uint32_t)p.tmem_cols) : "memory");
        asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
    }
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem_base = *s_tmem;
    const bool live = s_flag[2] != 0 && u1 > u0;

    if (warp == 0) {
        // ---------------- TMA producer ----------------
        if (lane == 0 && live) {
            asm volatile("prefetch.tensormap [%0];" ::"l"(&map_w) : "memory");
            asm volatile("prefetch.tensormap [%0];" ::"l"(&map_x) : "memory");
            asm volatile("prefetch.tensormap [%0];" ::"l"(&map_x64) : "memory");
            uint64_t pol_stream;
            asm volatile("createpolicy.fractional.L2::evict_first.b64 %0, 1.0;" : "=l"(pol_stream));
            // Weights do not depend on the previous kernel: fill the pipeline with W tiles first, then
            // wait for the previous kernel (which produces x) and add the x tiles of those stages.
            // This one thread feeds the whole pipeline, so its per-unit work is kept small: (tile, k block) advance
            // by increments (no 64-bit divisions), x comes in boxes of 64 rows where the pass has that many (one
            // request instead of four), and W is one bulk copy.
            const int n_units = (int)(u1 - u0);
            const int ahead = n_units < p.stages ? n_units : p.stages;
            const int tile0 = (int)(u0 / p.kb), kb0 = (int)(u0 % p.kb);
            auto load_x = [&](uint64_t* bar, uint8_t* sb, int kb) {
                int r = 0;
                for (; r + 64 <= p.rb; r += 64) tma_load_2d(&map_x64, bar, sb + r * 128, kb * WS_BK, p.row0 + r);
                for (; r < p.rb; r += 16) tma_load_2d(&map_x, bar, sb + r * 128, kb * WS_BK, p.row0 + r);
            };
            int tile = tile0, kb = kb0;
            for (int i = 0; i < ahead; ++i) {
                mbar_expect_tx(&full[i], stage_bytes);
                if (p.w_tiled) bulk_load_hint(base + (size_t)i * stage_bytes, p.w_tiled + (size_t)(u0 + i) * a_bytes, a_bytes, &full[i], pol_stream);
                else tma_load_2d_hint(&map_w, &full[i], base + (size_t)i * stage_bytes, kb * WS_BK, tile * WS_BM, pol_stream);
                if (++kb == p.kb) { kb = 0; ++tile; }
            }
            pdl_wait();
            if (blockIdx.x == 0) trace_mark(p.status, p.trace_kind);
            {
                int kbx = kb0;
                for (int i = 0; i < ahead; ++i) {
                    load_x(&full[i], base + (size_t)i * stage_bytes + a_bytes, kbx);
                    if (++kbx == p.kb) kbx = 0;
                }
            }
            int s = ahead == p.stages ? 0 : ahead;
            uint32_t ph = ahead == p.stages ? 1 : 0;
            const uint8_t* wsrc = p.w_tiled + (size_t)(u0 + ahead) * a_bytes;
            for (int i = ahead; i < n_units && !s_flag[0]; ++i) {
                if (!mbar_wait(&empty[s], ph ^ 1)) { s_flag[0] = 1; atomicCAS(p.status, 0, (int)ADED_ERR_TIMEOUT); break; }
                uint8_t* sa = base + (size_t)s * stage_bytes;
                mbar_expect_tx(&full[s], stage_bytes);
                if (p.w_tiled) bulk_load_hint(sa, wsrc, a_bytes, &full[s], pol_stream);
                else tma_load_2d_hint(&map_w, &full[s], sa, kb * WS_BK, tile * WS_BM, pol_stream);
                load_x(&full[s], sa + a_bytes, kb);
                wsrc += a_bytes;
                if (++kb == p.kb) { kb = 0; ++tile; }
                if (++s == p.stages) { s = 0; ph ^= 1; }
            }
        }
    } else if (warp == 1) {
        // ---------------- MMA issuer ----------------
        // The whole warp runs the loop and one elected lane issues: operands then stay warp-uniform.  An
        // instruction issued from a single-lane branch costs the issuing thread about 150 cycles on B200, an
        // elected one 30 to 60, and that time sits between a stage's arrival and its release.
        if (live) {
            const uint32_t idesc = (1u << 4) | (1u << 7) | (1u << 10) | ((uint32_t)(p.rb >> 3) << 17) | ((uint32_t)(WS_BM >> 4) << 24);
            const uint64_t desc0 = smem_desc_sw128(smem_u32(base));
            int s = 0;
            uint32_t ph = 0;
            int seg = 0;
            long long u = u0;
            bool ok = true;
            // (every exit from these loops is taken by the whole warp: the elected issue needs all 32 lanes)
            while (ok && u < u1 && !__any_sync(0xffffffffu, s_flag[0] != 0)) {
                const int kb0 = (int)(u % p.kb);
                long long ue = u + (p.kb - kb0);
                if (ue > u1) ue = u1;
                const int a = seg % p.n_acc;
                const uint32_t aph = (uint32_t)(seg / p.n_acc) & 1;
                if (!__all_sync(0xffffffffu, mbar_wait(&acc_empty[a], aph ^ 1))) { ok = false; break; }
                tc_fence_after();
                const uint32_t d_tmem = tmem_base + (uint32_t)(a * p.rb);
                bool first = true;
                for (; u < ue; ++u) {
                    if (!__all_sync(0xffffffffu, mbar_wait(&full[s], ph))) { ok = false; break; }
                    tc_fence_after();
                    const uint64_t da = desc0 + (uint64_t)(((uint32_t)s * stage_bytes) >> 4), db = da + (uint64_t)(a_bytes >> 4);
#pragma unroll
                    for (int kk = 0; kk < WS_BK / 16; ++kk) {
                        tc_mma_bf16_elect(d_tmem, da + (uint64_t)(kk * 2), db + (uint64_t)(kk * 2), idesc, first && kk == 0 ? 0u : 1u);
                    }
                    first = false;
                    tc_commit_elect(&empty[s]);      // stage reusable once these MMAs have read it
                    if (++s == p.stages) { s = 0; ph ^= 1; }
                }
                if (!ok) break;
                tc_commit_elect(&acc_full[a]);       // accumulator complete
                ++seg;
            }
            if (!ok && lane == 0) { s_flag[0] = 1; atomicCAS(p.status, 0, (int)ADED_ERR_TIMEOUT); }
        }
    } else {
        // ---------------- drain: warps 2..5, TMEM lane quarter = warp % 4 ----------------
        // Every segment's partial tile goes to slot (tile + CTA).
        const int quarter = warp & 3;
        const int row_in_tile = quarter * 32 + lane;           // W row inside the tile = TMEM lane
        int seg = 0;
        long long u = u0;
        while (live && u < u1) {
            const int tile = (int)(u / p.kb), kb0 = (int)(u % p.kb);
            long long ue = u + (p.kb - kb0);
            if (ue > u1) ue = u1;
            const int a = seg % p.n_acc;
            const uint32_t aph = (uint32_t)(seg / p.n_acc) & 1;
            if (!mbar_wait(&acc_full[a], aph)) { s_flag[0] = 1; atomicCAS(p.status, 0, (int)ADED_ERR_TIMEOUT); break; }
            tc_fence_after();
            const uint32_t taddr = tmem_base + ((uint32_t)(quarter * 32) << 16) + (uint32_t)(a * p.rb);
            float* slot = p.slots + (size_t)(tile + (int)blockIdx.x) * p.rb * WS_BM + row_in_tile;
            const bool slot_ok = ADED_IN_RANGE(tile >= 0 && tile < p.n_tiles && tile + (int)blockIdx.x < p.n_tiles + (int)gridDim.x, p.status);
            for (int c0 = 0; c0 < p.rb && slot_ok; c0 += 16) {
                float v[16];
                tc_ld16(taddr + (uint32_t)c0, v);
#pragma unroll
                for (int j = 0; j < 16; ++j) __stcg(slot + (size_t)(c0 + j) * WS_BM, v[j]);
            }
            tc_fence_before();
            __syncwarp();
            if (lane == 0) mbar_arrive(&acc_empty[a]);
            u = ue;
            ++seg;
        }
    }

    // ---------------- tail (LM head): per-row greedy candidates of the tiles this CTA contributed to ----------------
    // A tile's contributors are the consecutive CTAs whose unit ranges meet it.  Each publishes its partial
    // tiles (fence, then one arrival at every tile's counter), waits until all have arrived at its tiles,
    // and reduces a contiguous share of each tile's rows, a warp per row.
    tc_fence_before();
    __syncthreads();
    if (TAIL && u1 > u0) {
        // (A CTA that found the pass already failed when it started has computed nothing; it still arrives
        // at its counters, so that the others do not wait for it and the counts stay whole.)
        __shared__ int s_r0[WS_GMAX], s_item0[WS_GMAX + 1], s_ok;
        __shared__ TileRef s_tile[WS_GMAX];
        pdl_wait();                                  // (satisfied long ago; every thread now sees the previous kernels' writes)
        const bool store = live && *p.status == 0 && s_flag[0] == 0;
        const bool narrow = p.narrow != 0;
        const long long gu = p.kb;                   // units per tile
        const int g0 = (int)(u0 / gu), g1 = (int)((u1 - 1) / gu);
        __threadfence();
        __syncthreads();
        // arrive at every tile first: a CTA that waited at its first tile before announcing itself at its
        // second would chain the tiles of the whole launch one behind the other
        for (int g = g0 + (int)threadIdx.x; g <= g1; g += WS_THREADS)
            if (ws_owner_dev(g * gu, units, G, narrow) != ws_owner_dev((g + 1) * gu - 1, units, G, narrow)) ws_arrive(p.epi.counters + g);
        bool all_met = true;
        for (int gs = g0; gs <= g1 && all_met; gs += WS_GMAX) {
            const int ng = g1 - gs + 1 < WS_GMAX ? g1 - gs + 1 : WS_GMAX;
            if (threadIdx.x == 0) s_ok = 1;
            __syncthreads();
            if ((int)threadIdx.x < ng) {
                // one thread per tile: who contributes, this CTA's share of the rows, and the wait
                const int g = gs + (int)threadIdx.x;
                const int cf = ws_owner_dev(g * gu, units, G, narrow), cl = ws_owner_dev((g + 1) * gu - 1, units, G, narrow);
                const int n = cl - cf + 1, rank = (int)blockIdx.x - cf;
                const int r0 = rank * p.rows / n, r1 = (rank + 1) * p.rows / n;
                s_r0[threadIdx.x] = r0;
                s_item0[threadIdx.x + 1] = r1 - r0;
                s_tile[threadIdx.x] = p.epi.tiles[g];
                if (n > 1 && live && !ws_poll(p.epi.counters + g, (uint32_t)n * p.epi.epoch)) s_ok = 0;
            }
            __syncthreads();
            if (threadIdx.x == 0) {
                s_item0[0] = 0;
                for (int i = 0; i < ng; ++i) s_item0[i + 1] += s_item0[i];
            }
            __syncthreads();
            if (s_ok == 0) {
                if (threadIdx.x == 0) { s_flag[0] = 1; atomicCAS(p.status, 0, (int)ADED_ERR_TIMEOUT); }
                all_met = false;
            } else if (live) {
                const int total = s_item0[ng];
                for (int it = warp; it < total; it += WS_THREADS / 32) {
                    int gi = 0;
                    while (it >= s_item0[gi + 1]) ++gi;
                    ws_row_argmax(p, s_tile[gi], gs + gi, s_r0[gi] + it - s_item0[gi], lane, store);
                }
            }
            __syncthreads();
        }
    }

    // ---------------- teardown ----------------
    __syncthreads();
    if (warp == 0 && lane == 0 && s_flag[0]) {
        // unwinding after a timeout: give copies that are still in flight time to land (bounded)
        for (int i = 0; i < 1000; ++i) __nanosleep(1000);
    }
    __syncthreads();
    if (warp == 1) {
        tc_fence_after();
        asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem_base), "r"((uint32_t)p.tmem_cols) : "memory");
    }
}

// One warp runs the library's two kinds of bounded device-side wait on something that never happens -- an
// mbarrier nobody arrives at, an arrival counter nobody raises -- with a caller-chosen limit, and reports
// the outcome the way the kernels above do: ADED_ERR_TIMEOUT in the status word.  `which`: 0 mbarrier, 1 counter.
__global__ void k_wait_probe(int which, long long limit_cycles, const uint32_t* never_raised, int32_t* status) {
    __shared__ uint64_t bar;
    if (threadIdx.x == 0) {
        mbar_init(&bar, 1);
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    __syncwarp();
    bool ok;
    if (which == 0) ok = __all_sync(0xffffffffu, mbar_wait(&bar, 0, limit_cycles));
    else ok = ws_poll(never_raised, 0x40000000u, limit_cycles);
    if (!ok && threadIdx.x == 0) atomicCAS(status, 0, (int)ADED_ERR_TIMEOUT);
}

cudaError_t ws_wait_probe(int which, long long limit_cycles, const uint32_t* never_raised, int32_t* status, cudaStream_t st) {
    k_wait_probe<<<1, 32, 0, st>>>(which, limit_cycles, never_raised, status);
    return cudaGetLastError();
}

// W [n, k] row-major -> units of 128 rows x 64 columns, unit (tile, k block) at (tile * (k / 64) + k block) * 16 KB, each
// stored as the kernel stages it: row r at byte r * 128, its 16-byte chunk c at position c ^ (r & 7) (128-byte swizzle).
// A CTA's consecutive units are then one contiguous run of HBM.  One thread per 16-byte chunk.
__global__ void k_ws_retile(const uint4* __restrict__ w, uint4* __restrict__ out, int n, int k) {
    const size_t chunks = (size_t)n * k / 8;
    const int kb_n = k / WS_BK;
    for (size_t i = (size_t)blockIdx.x * blockDim.x + threadIdx.x; i < chunks; i += (size_t)gridDim.x * blockDim.x) {
        const size_t row = i / (k / 8);
        const int cc = (int)(i % (k / 8));                  // chunk within the row
        const int tile = (int)(row / WS_BM), r = (int)(row % WS_BM), kb = cc / 8, c = cc % 8;
        out[((size_t)tile * kb_n + kb) * (WS_BM * 8) + (size_t)r * 8 + (c ^ (r & 7))] = w[i];
    }
}

cudaError_t ws_retile(const void* w, void* out, int n, int k, cudaStream_t st) {
    k_ws_retile<<<2048, 256, 0, st>>>(static_cast<const uint4*>(w), static_cast<uint4*>(out), n, k);
    return cudaGetLastError();
}

// ---- host side --------------------------------------------------------------------------------
typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*,
                                  const cuuint64_t*, const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave,
                                  CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

static EncodeTiledFn encode_fn() {
    static EncodeTiledFn fn = nullptr;
    if (!fn) {
        void* p = nullptr;
        cudaDriverEntryPointQueryResult q;
        if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &p, cudaEnableDefault, &q) == cudaSuccess &&
            q == cudaDriverEntryPointSuccess)
            fn = reinterpret_cast<EncodeTiledFn>(p);
    }
    return fn;
}

// 2-D bf16 tensor [rows, cols] row-major, box = box_rows x 64 columns, 128-byte swizzle.
bool ws_make_map(CUtensorMap* map, const void* ptr, uint64_t rows, uint64_t cols, uint32_t box_rows) {
    EncodeTiledFn fn = encode_fn();
    if (!fn) return false;
    const cuuint64_t dims[2] = {cols, rows};
    const cuuint64_t strides[1] = {cols * 2};
    const cuuint32_t box[2] = {WS_BK, box_rows};
    const cuuint32_t elem[2] = {1, 1};
    return fn(map, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, const_cast<void*>(ptr), dims, strides, box, elem,
              CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
              CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

int ws_grid_limit(int device) {
    static int cached_dev = -1, cached = 0;
    if (cached_dev != device) {
        int sms = 0;
        cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, device);
        cached = 2 * sms;
        cached_dev = device;
    }
    return cached;
}

// CTAs a launch over n_tiles x kb units uses: two per SM, or one per SM (with twice the stages, so the same bytes
// in flight).  With one per SM a tile has half as many contributors, so the kernel that gathers the slots reads half
// as much; used where that kernel is the next thing on the critical path (see ws_one_per_sm in model.cu).
int ws_grid(int device, int n, int k, bool one_per_sm) {
    const long long units = (long long)(n / WS_BM) * (k / WS_BK);
    const int g = ws_grid_limit(device) / (one_per_sm ? 2 : 1);
    return units < g ? (int)units : g;
}

// Floats of slot storage for results of up to max_n columns and max_rows rows.
size_t ws_slot_floats(int device, int max_n, int max_rows) {
    const size_t passes = ((size_t)max_rows + 255) / 256;          // (regions of 256 rows also hold two regions of 128)
    return passes * ((size_t)max_n / WS_BM + ws_grid_limit(device)) * 256 * WS_BM;
}

// Raises the kernel's dynamic shared-memory limit; once per process, before any launch or capture.
bool ws_prepare() {
    return cudaFuncSetAttribute(k_gemm_ws<false>, cudaFuncAttributeMaxDynamicSharedMemorySize, 200 * 1024) == cudaSuccess &&
           cudaFuncSetAttribute(k_gemm_ws<true>, cudaFuncAttributeMaxDynamicSharedMemorySize, 112 * 1024) == cudaSuccess;
}

// Shapes the tensor-core path takes.
bool ws_supported(int n, int k) { return n % WS_BM == 0 && k % WS_BK == 0 && k >= WS_BK; }

// One pass: rows [row0, row0 + rows) of x (rows <= blk = 128 or 256) against all of W.  Partial tiles go to the
// slot region of pass row0 / blk; `epi` says whether the kernel's tail reduces them to greedy candidates.
cudaError_t ws_launch(const CUtensorMap& map_w, const void* w_tiled, const CUtensorMap& map_x, const CUtensorMap& map_x64, int rows, int row0, int blk,
                      int n, int k,
                      float* slots, int32_t* status, const WsEpilogue& epi, int trace_kind, int device, bool one_per_sm, cudaStream_t st) {
    WsParams p;
    p.w_tiled = static_cast<const uint8_t*>(w_tiled);
    p.rows = rows;
    p.rb = (rows + 15) / 16 * 16;
    p.row0 = row0;
    p.n = n;
    p.k = k;
    p.n_tiles = n / WS_BM;
    p.kb = k / WS_BK;
    const uint32_t stage_bytes = WS_BM * 128 + p.rb * 128;
    // About 100 KB per CTA: exactly two CTAs fit on an SM, so a launch of 2 x SMs CTAs is spread evenly
    // (a smaller footprint lets the scheduler stack three on some SMs and leave others empty); about 200 KB
    // for a launch of one CTA per SM.
    p.stages = (int)(((one_per_sm ? 200 : 100) * 1024) / stage_bytes);
    if (p.stages > 8) p.stages = 8;
    p.n_acc = p.rb > 128 ? 1 : 2;          // two CTAs per SM share 512 TMEM columns
    p.tmem_cols = 32;
    while (p.tmem_cols < p.n_acc * p.rb) p.tmem_cols *= 2;
    p.trace_kind = trace_kind;
    const int grid = ws_grid(device, n, k, one_per_sm);
    p.narrow = (long long)p.n_tiles * p.kb * (grid + 1) < (1ll << 31);
    p.slots = slots + (size_t)(row0 / blk) * (size_t)(p.n_tiles + grid) * blk * WS_BM;
    p.status = status;
    p.epi = epi;
    const size_t smem = (size_t)p.stages * stage_bytes + 1024 + 256;
    if (epi.mode == WS_EPI_ARGMAX) return launch_k(k_gemm_ws<true>, dim3(grid), dim3(WS_THREADS), smem, st, map_w, map_x, map_x64, p);
    return launch_k(k_gemm_ws<false>, dim3(grid), dim3(WS_THREADS), smem, st, map_w, map_x, map_x64, p);
}

}  // namespace aded
