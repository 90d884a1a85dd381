// One persistent kernel for a run of the decoder's projections together with the small steps
// between them ("forward pass through the model", Introduction):
//
//   GEMM_0 -> POST_0 -> GEMM_1 -> POST_1 -> ...        (up to FW_MAX_PAIRS pairs per launch)
//
// e.g.  O projection -> residual add + RMSNorm -> gate/up -> SwiGLU -> down -> residual add + RMSNorm
// of the next layer -> its QKV projection -> rotary embedding + K/V write.  Only the tree attention
// between two such runs is a kernel of its own.
//
// Why: launched one by one, every projection is followed by 5-7 us in which HBM is idle (the
// dependent kernel is released, gathers the partial tiles, stores its result, and the next GEMM is
// released in turn).  Here the CTAs stay resident, the steps are separated by grid-wide barriers
// (one atomic counter, bounded polling) and -- the point -- the TMA producer warp does not take
// part in them: weights do not depend on activations, so it keeps streaming the next projection's
// W tiles into the shared-memory ring while the other warps run the barrier and the small step.
// Only the x tiles of a stage wait for the step that produces x.
//
// Per CTA (192 threads, two CTAs per SM, grid = 2 x SMs; all CTAs are resident, which the barrier
// needs): warp 0 TMA producer, warp 1 MMA issuer (tcgen05, fp32 accumulators in TMEM, two of them),
// warps 2..5 epilogue and small steps.  GEMM work split, slots and contributor tables: gemm_out.cuh
// and gemm_ws.cu (same scheme).  The arithmetic of the small steps
// is that of dense_ws.cu.  Every wait is bounded; one that runs out raises ADED_ERR_TIMEOUT and the
// CTA unwinds (the others see the status word and unwind too).
#include <cuda.h>

#include <cstdio>
#include <cstdlib>

#include "aded_internal.cuh"
#include "fused_ws.cuh"
#include "gemm_out.cuh"
#include "tc_ptx.cuh"

namespace aded {

constexpr int FW_BM = 128, FW_BK = 64, FW_THREADS = 192, FW_EPI = 128;

__device__ __forceinline__ void epi_sync() { asm volatile("bar.sync 1, 128;" ::: "memory"); }   // warps 2..5
__device__ __forceinline__ uint32_t ld_acquire(const uint32_t* p) {
    uint32_t v;
    asm volatile("ld.acquire.gpu.global.u32 %0, [%1];" : "=r"(v) : "l"(p) : "memory");
    return v;
}
__device__ __forceinline__ void red_release(uint32_t* p) {
    asm volatile("red.release.gpu.global.add.u32 [%0], 1;" ::"l"(p) : "memory");
}
__device__ __forceinline__ void fence_async_global() { asm volatile("fence.proxy.async.global;" ::: "memory"); }

// Polls until the counter reaches `target`; false when the limit ran out or the pass has failed.
__device__ __forceinline__ bool counter_wait(const uint32_t* counter, uint32_t target, const int32_t* status) {
    const long long t0 = clock64();
    for (uint32_t spin = 0;; ++spin) {
        if (ld_acquire(counter) >= target) return true;
        if ((spin & 63) == 63) {
            if (*reinterpret_cast<const volatile int32_t*>(status) != 0) return false;
            if (clock64() - t0 > TC_WAIT_CYCLES) return false;
        }
        __nanosleep(32);
    }
}

// The epilogue warps leave their loops together: one thread samples the abort flag, all read the
// sample between two barriers (a warp that left alone would strand the others at a named barrier).
__device__ __forceinline__ bool epi_agree_abort(volatile int* flag, int et) {
    if (et == 0) flag[2] = flag[0];
    epi_sync();
    const bool a = flag[2] != 0;
    epi_sync();
    return a;
}

// ---- the small steps, run by the 128 epilogue threads of every CTA ---------------------------------
// Residual add + RMSNorm: CTA c owns row c.  Two sweeps over the row: the first adds the projection
// to the residual stream, stores it and sums the squares of the stored (rounded) values, the second
// reads the row back (this thread's own stores) and scales it.
__device__ __forceinline__ void post_add_norm(const FwParams& p, const GemmOut& y, const bf16* __restrict__ gain, int et,
                                              float* red) {
    const int r = blockIdx.x;
    if (r >= p.rows) return;            // uniform per CTA
    const int d = p.d;
    bf16* hrow = p.h + (size_t)r * d;
    float sq = 0.f;
#pragma unroll 4
    for (int c = et * 4; c < d; c += FW_EPI * 4) {
        const TileRef tr = y.tiles[c >> 7];
        uint2* hp = reinterpret_cast<uint2*>(hrow + c);
        const float4 hv = unpack4_bf16(*hp);
        const float4 add = gemm_out_at4(y, tr, r, c & 127);
        const uint2 nv = pack4_bf16(hv.x + add.x, hv.y + add.y, hv.z + add.z, hv.w + add.w);
        *hp = nv;
        const float4 v = unpack4_bf16(nv);
        sq += v.x * v.x + v.y * v.y + v.z * v.z + v.w * v.w;
    }
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) sq += __shfl_xor_sync(0xffffffffu, sq, o);
    if ((et & 31) == 0) red[et >> 5] = sq;
    epi_sync();
    const float total = red[0] + red[1] + red[2] + red[3];      // same order in every thread
    const float inv = rsqrtf(total / (float)d + p.eps);
#pragma unroll 4
    for (int c = et * 4; c < d; c += FW_EPI * 4) {
        const float4 v = unpack4_bf16(*reinterpret_cast<const uint2*>(hrow + c));
        const float4 g = unpack4_bf16(*reinterpret_cast<const uint2*>(gain + c));
        *reinterpret_cast<uint2*>(p.x + (size_t)r * d + c) = pack4_bf16(v.x * inv * g.x, v.y * inv * g.y, v.z * inv * g.z, v.w * inv * g.w);
    }
    epi_sync();                          // red[] may be reused
}

// act = round(silu(gate) * up), four columns per item, items spread over the grid.
__device__ __forceinline__ void post_swiglu(const FwParams& p, const GemmOut& gu, int et) {
    const int F = p.F, per_row = F >> 2;
    const long long items = (long long)p.rows * per_row;
    for (long long it = (long long)blockIdx.x * FW_EPI + et; it < items; it += (long long)gridDim.x * FW_EPI) {
        const int r = (int)(it / per_row), c = (int)(it % per_row) * 4;
        const TileRef tg = gu.tiles[c >> 7], tu = gu.tiles[(F + c) >> 7];
        const float4 g = gemm_out_at4(gu, tg, r, c & 127);
        const float4 u = gemm_out_at4(gu, tu, r, (F + c) & 127);
        *reinterpret_cast<uint2*>(p.act + (size_t)r * F + c) = swiglu4(g, u);
    }
}

// Rotary embedding + K/V write: item = (row, head, group of four rotary pairs).
__device__ __forceinline__ void post_rope_kv(const FwParams& p, const GemmOut& qkv, int layer, int et) {
    const int hd = p.hd, H = p.H, half = hd >> 1, d = p.d, gpr = half >> 2;     // groups per (row, head)
    const long long items = (long long)p.rows * H * gpr;
    for (long long it = (long long)blockIdx.x * FW_EPI + et; it < items; it += (long long)gridDim.x * FW_EPI) {
        const int i = (int)(it % gpr) * 4;
        const int hh = (int)((it / gpr) % H), r = (int)(it / ((long long)gpr * H));
        const int cq = hh * hd, ck = d + hh * hd, cv = 2 * d + hh * hd;
        const TileRef tq = qkv.tiles[cq >> 7], tk = qkv.tiles[ck >> 7], tv = qkv.tiles[cv >> 7];
        const int b = p.row_seq[r];
        const size_t slot = (size_t)p.kv_len[b] + p.row_local[r];
        const size_t cp = p.kv_cap[b];
        bf16* kdst = reinterpret_cast<bf16*>(p.kv_base[b]) + ((((size_t)layer * 2 + 0) * H + hh) * cp + slot) * hd;
        bf16* vdst = reinterpret_cast<bf16*>(p.kv_base[b]) + ((((size_t)layer * 2 + 1) * H + hh) * cp + slot) * hd;
        rope_kv_item(qkv, tq, tk, tv, r, cq, ck, cv, i, half, p.rope_cos + r * half, p.rope_sin + r * half, p.q + (size_t)r * d + hh * hd, kdst, vdst, true);
    }
}

// Work units of this CTA in one projection.  A projection with fewer units than CTAs is split over
// as many CTAs as it has units (the others idle), so that a tile's contributors are consecutive
// CTAs -- the same split, and the same contributor tables, as the stand-alone GEMM's.
__device__ __forceinline__ int fw_range(const FwPair& pr, long long G, long long& u0, long long& u1) {
    const long long units = (long long)pr.n_tiles * pr.kb;
    const long long g = units < G ? units : G;
    if ((long long)blockIdx.x < g) {
        u0 = ws_start(blockIdx.x, units, g);
        u1 = ws_start(blockIdx.x + 1, units, g);
    } else {
        u0 = u1 = 0;
    }
    return (int)g;
}

// x tiles of one stage: rb rows x 64 columns of the activation matrix, 16 rows per TMA box.
__device__ __forceinline__ void load_x_stage(const CUtensorMap* mx, uint64_t* bar, uint8_t* sb, int kb, int rb) {
    for (int r = 0; r < rb; r += 16) tma_load_2d(mx, bar, sb + r * 128, kb * FW_BK, r);
}

// Registers are capped at 112 per thread: the register file is handed out in units of four warps, so
// a CTA of six warps counts as eight, and at 128 registers (2 x 8 x 32 x 128 = the whole file) the
// occupancy query still reports one CTA per SM.
__global__ void __maxnreg__(112) k_fused_ws(const __grid_constant__ FwParams p) {
    extern __shared__ __align__(1024) uint8_t smem_raw[];
    uint8_t* base = (uint8_t*)(((uintptr_t)smem_raw + 1023) & ~(uintptr_t)1023);
    const uint32_t a_bytes = FW_BM * 128, b_bytes = (uint32_t)p.rb * 128, stage_bytes = a_bytes + b_bytes;
    uint64_t* bars = (uint64_t*)(base + (size_t)p.stages * stage_bytes);
    uint64_t* full = bars;
    uint64_t* empty = bars + p.stages;
    uint64_t* acc_full = bars + 2 * p.stages;
    uint64_t* acc_empty = acc_full + 2;
    uint32_t* s_tmem = (uint32_t*)(acc_empty + 2);
    volatile int* s_flag = (volatile int*)(s_tmem + 1);   // [0] abort, [1] pass had failed at entry, [2] abort as sampled for the epilogue warps
    float* s_red = (float*)(s_tmem + 4);

    pdl_launch_dependents();
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const long long G = gridDim.x;

    if (threadIdx.x == 0) {
        for (int s = 0; s < p.stages; ++s) { mbar_init(&full[s], 1); mbar_init(&empty[s], 1); }
        for (int a = 0; a < 2; ++a) { mbar_init(&acc_full[a], 1); mbar_init(&acc_empty[a], 4); }
        s_flag[0] = 0;
        s_flag[1] = *p.status != 0;
        s_flag[2] = 0;
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
    const bool live = s_flag[1] == 0;      // a pass that has already failed does nothing

    if (warp == 0) {
        // ---------------- TMA producer: streams W ahead of the barriers, adds x when it exists ----------------
        if (lane == 0 && live) {
            uint64_t pol_stream;
            asm volatile("createpolicy.fractional.L2::evict_first.b64 %0, 1.0;" : "=l"(pol_stream));
            long long issued = 0;            // stages filled so far, over all projections
            int pend_stage[8], pend_kb[8];   // newest stages that hold W but not yet x
            int pending = 0;
            for (int i = 0; i < p.n_pairs && !s_flag[0]; ++i) {
                const FwPair& pr = p.pair[i];
                const CUtensorMap* mw = p.maps + pr.map_w;
                const CUtensorMap* mx = p.maps + pr.map_x;
                asm volatile("prefetch.tensormap [%0];" ::"l"(mw) : "memory");
                asm volatile("prefetch.tensormap [%0];" ::"l"(mx) : "memory");
                long long u0, u1;
                fw_range(pr, G, u0, u1);
                // x of projection i exists once the step before it has finished on every CTA: for the
                // first projection that is the previous kernel, afterwards i G arrivals at the counter
                // of finished steps.  (Steps and projections count separately: a CTA without work in a
                // projection arrives at its barrier at once, and one shared count could reach the target
                // while another CTA is still inside the step.)
                const uint32_t target = (uint32_t)(i * G);
                bool x_ready = false;
                for (long long u = u0; u <= u1 && !s_flag[0]; ++u) {
                    const bool last = u == u1;          // one extra round that only settles the pending stages
                    if (!x_ready && (pending > 0 || !last)) {
                        const bool must = pending == p.stages || last;
                        bool ok = false;
                        if (i == 0) {
                            if (must) { pdl_wait(); ok = true; }
                        } else if (must) {
                            ok = counter_wait(p.counter + 1, target, p.status);
                            if (!ok) { s_flag[0] = 1; atomicCAS(p.status, 0, (int)ADED_ERR_TIMEOUT); break; }
                        } else {
                            ok = ld_acquire(p.counter + 1) >= target;
                        }
                        if (ok) {
                            fence_async_global();
                            for (int j = 0; j < pending; ++j)
                                load_x_stage(mx, &full[pend_stage[j]], base + (size_t)pend_stage[j] * stage_bytes + a_bytes, pend_kb[j], p.rb);
                            pending = 0;
                            x_ready = true;
                        }
                    }
                    if (last) break;
                    const int s = (int)(issued % p.stages);
                    if (issued >= p.stages) {
                        const uint32_t par = (uint32_t)((issued / p.stages - 1) & 1);
                        if (!mbar_wait(&empty[s], par)) { s_flag[0] = 1; atomicCAS(p.status, 0, (int)ADED_ERR_TIMEOUT); break; }
                    }
                    const int tile = (int)(u / pr.kb), kb = (int)(u % pr.kb);
                    uint8_t* sa = base + (size_t)s * stage_bytes;
                    mbar_expect_tx(&full[s], stage_bytes);
                    tma_load_2d_hint(mw, &full[s], sa, kb * FW_BK, tile * FW_BM, pol_stream);
                    if (x_ready) {
                        load_x_stage(mx, &full[s], sa + a_bytes, kb, p.rb);
                    } else {
                        pend_stage[pending] = s;
                        pend_kb[pending] = kb;
                        ++pending;
                    }
                    ++issued;
                }
            }
        }
    } else if (warp == 1) {
        // ---------------- MMA issuer ----------------
        if (lane == 0 && live) {
            const uint32_t idesc = (1u << 4) | (1u << 7) | (1u << 10) | ((uint32_t)(p.rb >> 3) << 17) | ((uint32_t)(FW_BM >> 4) << 24);
            long long consumed = 0;
            int seg = 0;
            for (int i = 0; i < p.n_pairs && !s_flag[0]; ++i) {
                const FwPair& pr = p.pair[i];
                long long u0, u1;
                fw_range(pr, G, u0, u1);
                long long u = u0;
                while (u < u1 && !s_flag[0]) {
                    const int kb0 = (int)(u % pr.kb);
                    long long ue = u + (pr.kb - kb0);
                    if (ue > u1) ue = u1;
                    const int a = seg & 1;
                    const uint32_t aph = (uint32_t)(seg >> 1) & 1;
                    if (!mbar_wait(&acc_empty[a], aph ^ 1)) { s_flag[0] = 1; atomicCAS(p.status, 0, (int)ADED_ERR_TIMEOUT); break; }
                    tc_fence_after();
                    const uint32_t d_tmem = tmem_base + (uint32_t)(a * p.rb);
                    bool first = true;
                    for (; u < ue; ++u) {
                        const int s = (int)(consumed % p.stages);
                        if (!mbar_wait(&full[s], (uint32_t)((consumed / p.stages) & 1))) {
                            s_flag[0] = 1;
                            atomicCAS(p.status, 0, (int)ADED_ERR_TIMEOUT);
                            break;
                        }
                        tc_fence_after();
                        const uint32_t sa = smem_u32(base + (size_t)s * stage_bytes);
                        const uint64_t da = smem_desc_sw128(sa), db = smem_desc_sw128(sa + a_bytes);
#pragma unroll
                        for (int kk = 0; kk < FW_BK / 16; ++kk)
                            tc_mma_bf16(d_tmem, da + (uint64_t)(kk * 2), db + (uint64_t)(kk * 2), idesc, first && kk == 0 ? 0u : 1u);
                        first = false;
                        tc_commit(&empty[s]);
                        ++consumed;
                    }
                    if (s_flag[0]) break;
                    tc_commit(&acc_full[a]);
                    ++seg;
                }
            }
        }
    } else if (warp < 6) {
        // ---------------- epilogue and small steps: warps 2..5 ----------------
        const int quarter = warp & 3;
        const int row_in_tile = quarter * 32 + lane;
        const int et = threadIdx.x - 64;
        int seg = 0;
        // These warps read and write activations of earlier kernels: wait for them, then look at the
        // status word again (a failed tree check may have been written after this CTA started).
        pdl_wait();
        if (et == 0 && *reinterpret_cast<const volatile int32_t*>(p.status) != 0) s_flag[0] = 1;
        for (int i = 0; i < p.n_pairs && live; ++i) {
            if (epi_agree_abort(s_flag, et)) break;
            const FwPair& pr = p.pair[i];
            long long u0, u1;
            const int g_eff = fw_range(pr, G, u0, u1);
            long long u = u0;
            while (u < u1) {
                const int tile = (int)(u / pr.kb), kb0 = (int)(u % pr.kb);
                long long ue = u + (pr.kb - kb0);
                if (ue > u1) ue = u1;
                const int a = seg & 1;
                const uint32_t aph = (uint32_t)(seg >> 1) & 1;
                if (!mbar_wait(&acc_full[a], aph)) { s_flag[0] = 1; atomicCAS(p.status, 0, (int)ADED_ERR_TIMEOUT); break; }
                tc_fence_after();
                const uint32_t taddr = tmem_base + ((uint32_t)(quarter * 32) << 16) + (uint32_t)(a * p.rb);
                float* slot = p.slots + (size_t)(tile + (int)blockIdx.x) * p.rb * FW_BM + row_in_tile;
                for (int c0 = 0; c0 < p.rb; c0 += 16) {
                    float v[16];
                    tc_ld16(taddr + (uint32_t)c0, v);
#pragma unroll
                    for (int j = 0; j < 16; ++j) __stcg(slot + (size_t)(c0 + j) * FW_BM, v[j]);
                }
                tc_fence_before();
                __syncwarp();
                if (lane == 0) mbar_arrive(&acc_empty[a]);
                u = ue;
                ++seg;
            }
            if (pr.post == FW_POST_NONE) continue;     // only the last projection of a launch: the kernel's end publishes it
            // every CTA's partial tiles of projection i are in memory ...
            __threadfence();
            epi_sync();
            if (et == 0) {
                if (!s_flag[0]) {
                    red_release(p.counter);
                    if (!counter_wait(p.counter, (uint32_t)((i + 1) * G), p.status)) {
                        s_flag[0] = 1;
                        atomicCAS(p.status, 0, (int)ADED_ERR_TIMEOUT);
                    }
                }
            }
            if (epi_agree_abort(s_flag, et)) break;
            // ... the step that consumes them ...
            GemmOut o;
            o.y = nullptr;
            o.slots = p.slots;
            o.tiles = pr.tiles;
            o.mode = 1;
            o.n = pr.n_tiles * FW_BM;
            o.n_tiles = pr.n_tiles;
            o.kb = pr.kb;
            o.g = g_eff;
            o.rows = p.rows;
            if (pr.post == FW_POST_ADD_NORM) post_add_norm(p, o, reinterpret_cast<const bf16*>(pr.gain), et, s_red);
            else if (pr.post == FW_POST_SWIGLU) post_swiglu(p, o, et);
            else post_rope_kv(p, o, pr.layer, et);
            // ... and its result is in memory for the next projection's TMA loads
            __threadfence();
            fence_async_global();
            epi_sync();
            if (et == 0) red_release(p.counter + 1);
        }
    }

    // ---------------- teardown ----------------
    tc_fence_before();
    __syncthreads();
    if (warp == 0 && lane == 0 && s_flag[0]) {
        for (int i = 0; i < 1000; ++i) __nanosleep(1000);   // unwinding: let copies in flight land (bounded)
    }
    __syncthreads();
    if (warp == 1) {
        tc_fence_after();
        asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem_base), "r"((uint32_t)p.tmem_cols) : "memory");
    }
}

// ---- host side --------------------------------------------------------------------------------------
static size_t fw_smem(int rb, int* stages_out) {
    const uint32_t stage_bytes = FW_BM * 128 + rb * 128;
    int stages = (int)((100 * 1024) / stage_bytes);      // about 100 KB: exactly two CTAs per SM
    if (stages > 8) stages = 8;
    if (stages_out) *stages_out = stages;
    return (size_t)stages * stage_bytes + 1024 + 256;
}

// The grid barrier needs every CTA resident: two per SM must fit.  The runtime's occupancy query
// answers one CTA per SM for this kernel whatever block size and shared memory are asked about (it
// seems not to model kernels that allocate tensor memory), so the check is done by hand from the
// device's limits: registers are granted per group of four warps, shared memory per CTA plus the
// reserved kilobyte, tensor memory 512 columns per SM.
bool fw_prepare(int device) {
    if (cudaFuncSetAttribute(k_fused_ws, cudaFuncAttributeMaxDynamicSharedMemorySize, 112 * 1024) != cudaSuccess) {
        cudaGetLastError();
        return false;
    }
    cudaFuncAttributes fa = {};
    if (cudaFuncGetAttributes(&fa, k_fused_ws) != cudaSuccess) { cudaGetLastError(); return false; }
    int regs_sm = 0, smem_sm = 0, smem_res = 0, threads_sm = 0;
    cudaDeviceGetAttribute(&regs_sm, cudaDevAttrMaxRegistersPerMultiprocessor, device);
    cudaDeviceGetAttribute(&smem_sm, cudaDevAttrMaxSharedMemoryPerMultiprocessor, device);
    cudaDeviceGetAttribute(&smem_res, cudaDevAttrReservedSharedMemoryPerBlock, device);
    cudaDeviceGetAttribute(&threads_sm, cudaDevAttrMaxThreadsPerMultiProcessor, device);
    const int warps = (FW_THREADS / 32 + 3) / 4 * 4;
    const long long regs_cta = (long long)warps * 32 * ((fa.numRegs + 7) / 8 * 8);
    const long long smem_cta = (long long)fw_smem(128, nullptr) + fa.sharedSizeBytes + smem_res;
    const bool ok = 2 * regs_cta < regs_sm && 2 * smem_cta <= smem_sm && 2 * FW_THREADS <= threads_sm;
    if (getenv("ADED_VERBOSE"))
        fprintf(stderr, "[aded] persistent projection kernel: %d registers, %lld of %d registers and %lld of %d bytes of shared memory for two CTAs: %s\n",
                fa.numRegs, 2 * regs_cta, regs_sm, 2 * smem_cta, smem_sm, ok ? "used" : "not used");
    return ok;
}

cudaError_t fw_launch(aded_model* m, aded_kv* kv, const FwPair* pairs, int n_pairs, int rows, int launch_index, cudaStream_t st) {
    FwParams p = {};
    p.n_pairs = n_pairs;
    for (int i = 0; i < n_pairs; ++i) p.pair[i] = pairs[i];
    p.rows = rows;
    p.rb = (rows + 15) / 16 * 16;
    const size_t smem = fw_smem(p.rb, &p.stages);
    p.tmem_cols = 32;
    while (p.tmem_cols < 2 * p.rb) p.tmem_cols *= 2;
    p.maps = m->fw_maps;
    p.slots = m->ws_slots;
    p.counter = m->fw_counters + 2 * (launch_index % FW_COUNTERS);
    p.status = m->status;
    p.h = (bf16*)m->h;
    p.x = (bf16*)m->x;
    p.q = (bf16*)m->q;
    p.act = (bf16*)m->act;
    p.d = m->cfg.d_model;
    p.F = m->cfg.d_ffn;
    p.H = m->cfg.n_heads;
    p.hd = m->cfg.head_dim;
    p.eps = m->cfg.rms_eps;
    p.rope_cos = m->rope_cos;
    p.rope_sin = m->rope_sin;
    p.kv_base = (char* const*)kv->base_dev;
    p.kv_cap = kv->cap_dev;
    p.kv_len = kv->len_dev;
    p.row_seq = m->rows.seq;
    p.row_local = m->rows.local;
    return launch_k(k_fused_ws, dim3(ws_grid_limit(m->device)), dim3(FW_THREADS), smem, st, p);
}

}  // namespace aded
