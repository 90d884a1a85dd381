// Tree attention on the 5th-generation tensor cores (bf16 models, head_dim 128).
//
// Same computation and the same rounding as k_tree_attn_mma (tree_attention.cu): every tree node
// attends to all committed cache positions and to its ancestors and itself ("Draft Construction and
// Verification"), scores in the log2 domain against an integer running reference, numerators rounded
// to bf16 for the P V product, row sums unrounded.  What differs is where the work runs:
//   * a CTA owns (sequence, head, key split, block of 64 query rows); the key splits of one
//     (sequence, head, row block) form a thread-block cluster and are merged through distributed
//     shared memory exactly as in the mma.sync kernel;
//   * warp 0 streams 64-key blocks of K and V with TMA (two boxes of 64 x 64 per block, 128-byte
//     swizzle) into two stages each; warp 1 issues tcgen05.mma; warps 2..5 run the softmax;
//   * S = Q K^T: M = 64 (query rows), N = 64 (the block's keys), K = 128: 8 instructions.  An M = 64
//     accumulator occupies lanes 0..15 of each of the four TMEM lane quarters.  A softmax warp reads
//     it with the 16-lane load whose second half-warp takes the same lanes 32 columns further
//     (16x32bx2): thread (lane & 15) + 16 * quarter is the query row, lane >> 4 the key half, 32 scores
//     per thread.  A row's two threads sit in the same warp and share the row maximum with one
//     shuffle; nothing else crosses threads;
//   * O += P V: M = 64, N = 128 (head_dim), K = 64 keys: 4 instructions.  P (bf16) is written by the
//     softmax warps into a K-major swizzled tile, V is used as stored (keys x head_dim, i.e. MN-major
//     B operand whose two 64-element halves are one sub-tile apart); a thread owns half a row of O
//     (the same split load, 64 columns apart).  O stays in TMEM over all blocks; when a row's
//     reference moves (rare: it is an integer) its owner rescales its part in place;
//   * all S/P/O hand-overs go through mbarriers (tcgen05.commit on the MMA side); every wait is
//     bounded and a wait that runs out raises ADED_ERR_TIMEOUT, after which the CTA still takes part
//     in the cluster's barriers and frees its TMEM.
// Rows of the cache past the last key are read by the last block's TMA box and must be finite (their
// probabilities are exactly zero): the cache is zero-filled when it is created and only ever
// receives K/V rows, so they are.
#include <cuda.h>

#include "aded_internal.cuh"
#include "tc_ptx.cuh"

namespace aded {

constexpr int AT_BLK = 64;        // keys per block
constexpr int AT_ROWS = 64;       // query rows per CTA
constexpr int AT_HD = 128;
constexpr int AT_STAGES = 2;      // K and V blocks in flight
constexpr int AT_THREADS = 192;
constexpr int AT_TMEM_COLS = 256; // S: 2 x 64, O: 128 (lanes 0..15 of every lane quarter)
constexpr uint32_t AT_S_COL = 0, AT_O_COL = 128;
constexpr float AT_SLACK = 8.f;   // how far a row's maximum may exceed its reference (log2 domain) before O is rescaled
constexpr uint32_t AT_SUB = 64 * 128;            // bytes of a 64-row x 128-byte sub-tile
// shared-memory map (from a 1024-byte aligned base)
constexpr uint32_t AT_OFF_Q = 0;                                   // 2 sub-tiles (head_dim halves)
constexpr uint32_t AT_OFF_P = AT_OFF_Q + 2 * AT_SUB;               // 2 buffers
constexpr uint32_t AT_OFF_K = AT_OFF_P + 2 * AT_SUB;               // stages x 2 sub-tiles
constexpr uint32_t AT_OFF_V = AT_OFF_K + AT_STAGES * 2 * AT_SUB;   // stages x 2 sub-tiles
constexpr uint32_t AT_OFF_BAR = AT_OFF_V + AT_STAGES * 2 * AT_SUB;
constexpr uint32_t AT_SMEM = AT_OFF_BAR + 256 + 1024;
// merge scratch over the K stages (free once every MMA has completed)
constexpr uint32_t AT_OFF_SO = AT_OFF_K;                           // [64][128] fp32, float4 index swizzled by row
constexpr uint32_t AT_OFF_SML = AT_OFF_V;                          // [64][2] fp32

struct AttnTcArgs {
    const CUtensorMap* kv_maps;    // [batch] device array: 3-D maps (head_dim, capacity, layer x {K,V} x head)
    bf16* out;                     // [R][H][HD]
    const int32_t* len;
    const int32_t* row_off;
    const uint64_t* anc;
    int layer, H, n_splits, row_blocks;
    float scale_log2;
    int32_t* status;
};

__device__ __forceinline__ void tma_load_3d(const CUtensorMap* map, uint64_t* bar, void* dst, int c0, int c1, int c2) {
    asm volatile(
        "cp.async.bulk.tensor.3d.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%3, %4, %5}], [%2];"
        ::"r"(smem_u32(dst)), "l"(map), "r"(smem_u32(bar)), "r"(c0), "r"(c1), "r"(c2) : "memory");
}

__device__ __forceinline__ void tma_prefetch_3d(const CUtensorMap* map, int c0, int c1, int c2) {
    asm volatile("cp.async.bulk.prefetch.tensor.3d.L2.global.tile [%0, {%1, %2, %3}];" ::"l"(map), "r"(c0), "r"(c1), "r"(c2) : "memory");
}

// 32 consecutive fp32 columns of this warp's 32 TMEM lanes.
__device__ __forceinline__ void tc_ld32(uint32_t taddr, uint32_t* r) {
    asm volatile(
        "tcgen05.ld.sync.aligned.32x32b.x32.b32 {%0, %1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15, "
        "%16, %17, %18, %19, %20, %21, %22, %23, %24, %25, %26, %27, %28, %29, %30, %31}, [%32];"
        : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7]),
          "=r"(r[8]), "=r"(r[9]), "=r"(r[10]), "=r"(r[11]), "=r"(r[12]), "=r"(r[13]), "=r"(r[14]), "=r"(r[15]),
          "=r"(r[16]), "=r"(r[17]), "=r"(r[18]), "=r"(r[19]), "=r"(r[20]), "=r"(r[21]), "=r"(r[22]), "=r"(r[23]),
          "=r"(r[24]), "=r"(r[25]), "=r"(r[26]), "=r"(r[27]), "=r"(r[28]), "=r"(r[29]), "=r"(r[30]), "=r"(r[31])
        : "r"(taddr) : "memory");
    asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory");
}
__device__ __forceinline__ void tc_st32(uint32_t taddr, const uint32_t* r) {
    asm volatile(
        "tcgen05.st.sync.aligned.32x32b.x32.b32 [%32], {%0, %1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15, "
        "%16, %17, %18, %19, %20, %21, %22, %23, %24, %25, %26, %27, %28, %29, %30, %31};"
        ::"r"(r[0]), "r"(r[1]), "r"(r[2]), "r"(r[3]), "r"(r[4]), "r"(r[5]), "r"(r[6]), "r"(r[7]),
          "r"(r[8]), "r"(r[9]), "r"(r[10]), "r"(r[11]), "r"(r[12]), "r"(r[13]), "r"(r[14]), "r"(r[15]),
          "r"(r[16]), "r"(r[17]), "r"(r[18]), "r"(r[19]), "r"(r[20]), "r"(r[21]), "r"(r[22]), "r"(r[23]),
          "r"(r[24]), "r"(r[25]), "r"(r[26]), "r"(r[27]), "r"(r[28]), "r"(r[29]), "r"(r[30]), "r"(r[31]),
          "r"(taddr) : "memory");
    asm volatile("tcgen05.wait::st.sync.aligned;" ::: "memory");
}

// MN-major operand tile (rows = k index, 128-byte lines of 64 m/n elements, 128-byte swizzle): groups of
// eight k rows 1024 bytes apart; a second 64-element column of the m/n extent would be `lbo` bytes away.
__device__ __forceinline__ uint64_t smem_desc_mn_sw128(uint32_t addr, uint32_t lbo) {
    uint64_t d = 0;
    d |= (uint64_t)((addr & 0x3FFFF) >> 4);
    d |= (uint64_t)((lbo >> 4) & 0x3FFF) << 16;
    d |= (uint64_t)(1024 >> 4) << 32;
    d |= (uint64_t)1 << 46;
    d |= (uint64_t)2 << 61;
    return d;
}

// 32 fp32 columns of lanes 0..15 of this warp's TMEM lane quarter: threads 0..15 get columns c .. c + 31 of
// lane `thread`, threads 16..31 the columns SPLIT further of lane `thread - 16`.
template <int SPLIT>
__device__ __forceinline__ void tc_ld32_split(uint32_t taddr, uint32_t* r) {
    asm volatile(
        "tcgen05.ld.sync.aligned.16x32bx2.x32.b32 {%0, %1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15, "
        "%16, %17, %18, %19, %20, %21, %22, %23, %24, %25, %26, %27, %28, %29, %30, %31}, [%32], %33;"
        : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7]),
          "=r"(r[8]), "=r"(r[9]), "=r"(r[10]), "=r"(r[11]), "=r"(r[12]), "=r"(r[13]), "=r"(r[14]), "=r"(r[15]),
          "=r"(r[16]), "=r"(r[17]), "=r"(r[18]), "=r"(r[19]), "=r"(r[20]), "=r"(r[21]), "=r"(r[22]), "=r"(r[23]),
          "=r"(r[24]), "=r"(r[25]), "=r"(r[26]), "=r"(r[27]), "=r"(r[28]), "=r"(r[29]), "=r"(r[30]), "=r"(r[31])
        : "r"(taddr), "n"(SPLIT) : "memory");
    asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory");
}
template <int SPLIT>
__device__ __forceinline__ void tc_st32_split(uint32_t taddr, const uint32_t* r) {
    asm volatile(
        "tcgen05.st.sync.aligned.16x32bx2.x32.b32 [%32], %33, {%0, %1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15, "
        "%16, %17, %18, %19, %20, %21, %22, %23, %24, %25, %26, %27, %28, %29, %30, %31};"
        ::"r"(r[0]), "r"(r[1]), "r"(r[2]), "r"(r[3]), "r"(r[4]), "r"(r[5]), "r"(r[6]), "r"(r[7]),
          "r"(r[8]), "r"(r[9]), "r"(r[10]), "r"(r[11]), "r"(r[12]), "r"(r[13]), "r"(r[14]), "r"(r[15]),
          "r"(r[16]), "r"(r[17]), "r"(r[18]), "r"(r[19]), "r"(r[20]), "r"(r[21]), "r"(r[22]), "r"(r[23]),
          "r"(r[24]), "r"(r[25]), "r"(r[26]), "r"(r[27]), "r"(r[28]), "r"(r[29]), "r"(r[30]), "r"(r[31]),
          "r"(taddr), "n"(SPLIT) : "memory");
    asm volatile("tcgen05.wait::st.sync.aligned;" ::: "memory");
}

// Bounded wait that also gives up when another thread of the CTA has raised the abort flag.
__device__ __forceinline__ bool at_wait(uint64_t* bar, uint32_t parity, volatile int* abort_flag) {
    const uint32_t addr = smem_u32(bar);
    const long long t0 = clock64();
    for (uint32_t spin = 0;; ++spin) {
        uint32_t done;
        asm volatile(
            "{\n\t.reg .pred p;\n\t"
            "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\t"
            "selp.u32 %0, 1, 0, p;\n\t}"
            : "=r"(done) : "r"(addr), "r"(parity) : "memory");
        if (done) return true;
        if ((spin & 255) == 255 && (*abort_flag || clock64() - t0 > TC_WAIT_CYCLES)) return false;
    }
}

__device__ __forceinline__ float at_ex2(float x) {
    float y;
    asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
    return y;
}
__device__ __forceinline__ uint32_t at_pack(float lo, float hi) {
    __nv_bfloat162 v = __floats2bfloat162_rn(lo, hi);
    return *reinterpret_cast<uint32_t*>(&v);
}

__global__ void __launch_bounds__(AT_THREADS, 2)
k_tree_attn_tc(const __grid_constant__ CUtensorMap map_q, AttnTcArgs a) {
    extern __shared__ __align__(1024) uint8_t smem_raw[];
    uint8_t* base = (uint8_t*)(((uintptr_t)smem_raw + 1023) & ~(uintptr_t)1023);
    uint64_t* bars = (uint64_t*)(base + AT_OFF_BAR);
    uint64_t* q_full = bars;
    uint64_t* k_full = bars + 1;
    uint64_t* k_empty = bars + 3;
    uint64_t* v_full = bars + 5;
    uint64_t* v_empty = bars + 7;
    uint64_t* s_full = bars + 9;
    uint64_t* s_empty = bars + 11;
    uint64_t* p_full = bars + 13;
    uint64_t* p_empty = bars + 15;
    uint32_t* s_tmem = (uint32_t*)(bars + 17);
    volatile int* s_flag = (volatile int*)(s_tmem + 2);     // [0] abort
    volatile int* s_off = s_flag + 2;                       // [stage] 1: the stage's full barriers are one phase ahead

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    if (threadIdx.x == 0) {
        mbar_init(q_full, 1);
        for (int i = 0; i < 2; ++i) {
            mbar_init(&k_full[i], 1); mbar_init(&k_empty[i], 1);
            mbar_init(&v_full[i], 1); mbar_init(&v_empty[i], 1);
            mbar_init(&s_full[i], 1); mbar_init(&s_empty[i], 4);
            mbar_init(&p_full[i], 4); mbar_init(&p_empty[i], 1);
        }
        s_flag[0] = 0;
        s_off[0] = 0;
        s_off[1] = 0;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
        asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
    }
    if (warp == 1) {
        asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(s_tmem)), "r"((uint32_t)AT_TMEM_COLS) : "memory");
        asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
    }
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem_base = *s_tmem;
    // Only now may the next kernel's blocks appear: every block of this kernel holds its tensor memory,
    // so a later kernel's allocation can make none of them wait.
    pdl_launch_dependents();
    // While the previous kernel (which writes q and the tree's own K/V rows) is still running, the
    // producer already fetches this CTA's first two key blocks into their stages, if they lie entirely in
    // the committed part of the cache (which no kernel of the pass writes), and asks L2 for the others.
    // The committed length and the tree size are read on trust here; both are read again after the wait
    // and the early blocks are used only if the two reads agree, otherwise they are fetched again.
    int n_pre = 0, pre_L = -1, pre_T = -1;
    if (warp == 0 && lane == 0) {
        const int pb = blockIdx.z / a.row_blocks;
        const CUtensorMap* kvm = a.kv_maps + pb;
        asm volatile("prefetch.tensormap [%0];" ::"l"(&map_q) : "memory");
        asm volatile("prefetch.tensormap [%0];" ::"l"(kvm) : "memory");
        pre_L = __ldcg(a.len + pb);
        pre_T = __ldcg(a.row_off + pb + 1) - __ldcg(a.row_off + pb);
        if (pre_L >= 0 && pre_T >= 1 && pre_T <= ADED_MAX_NODES && pre_L < (1 << 28)) {
            const int pnb = (pre_L + pre_T + AT_BLK - 1) / AT_BLK;
            const int b0 = (int)((long long)blockIdx.y * pnb / a.n_splits);
            int b1 = (int)((long long)(blockIdx.y + 1) * pnb / a.n_splits);
            if (b1 > b0 + 32) b1 = b0 + 32;
            const int plane_k = (a.layer * 2 + 0) * a.H + blockIdx.x, plane_v = (a.layer * 2 + 1) * a.H + blockIdx.x;
            for (int blk = b0; blk < b1; ++blk) {
                const int j = blk - b0, key0 = blk * AT_BLK;
                if (j < AT_STAGES && n_pre == j && key0 + AT_BLK <= pre_L) {
                    uint8_t* dk = base + AT_OFF_K + (uint32_t)j * 2 * AT_SUB;
                    uint8_t* dv = base + AT_OFF_V + (uint32_t)j * 2 * AT_SUB;
                    mbar_expect_tx(&k_full[j], 2 * AT_SUB);
                    tma_load_3d(kvm, &k_full[j], dk, 0, key0, plane_k);
                    tma_load_3d(kvm, &k_full[j], dk + AT_SUB, 64, key0, plane_k);
                    mbar_expect_tx(&v_full[j], 2 * AT_SUB);
                    tma_load_3d(kvm, &v_full[j], dv, 0, key0, plane_v);
                    tma_load_3d(kvm, &v_full[j], dv + AT_SUB, 64, key0, plane_v);
                    ++n_pre;
                } else {
                    tma_prefetch_3d(kvm, 0, key0, plane_k);
                    tma_prefetch_3d(kvm, 64, key0, plane_k);
                    tma_prefetch_3d(kvm, 0, key0, plane_v);
                    tma_prefetch_3d(kvm, 64, key0, plane_v);
                }
            }
        }
    }
    pdl_wait();
    if (first_thread_of_grid()) trace_mark(a.status, TK_ATTN);
    const int pass_status = *a.status;

    const int hh = blockIdx.x, split = blockIdx.y, b = blockIdx.z / a.row_blocks;
    const int row_base = (blockIdx.z % a.row_blocks) * AT_ROWS;     // first query row (node of the tree) of this CTA
    const int off = a.row_off[b];
    const int T = a.row_off[b + 1] - off;
    const int L = __ldcg(a.len + b);
    const int n_keys = L + T;
    const int nb = (n_keys + AT_BLK - 1) / AT_BLK;
    const int blk0 = (int)((long long)split * nb / a.n_splits);
    const int blk1 = (int)((long long)(split + 1) * nb / a.n_splits);
    // A failed pass does no work here but still takes part in the cluster's barriers below.
    const int nblk = pass_status == 0 ? blk1 - blk0 : 0;

    if (warp == 0) {
        // ---------------- TMA producer ----------------
        if (lane == 0) {
            bool ok = true;
            if (n_pre > 0 && (L != pre_L || T != pre_T || nblk < n_pre)) {
                // The early reads were stale (or the pass has failed): let the early copies land; the stages
                // are then filled again, in the next phase of their barriers (s_off tells the consumers).
                for (int j = 0; j < n_pre; ++j) {
                    ok = ok && at_wait(&k_full[j], 0, s_flag) && at_wait(&v_full[j], 0, s_flag);
                    s_off[j] = 1;
                }
                n_pre = 0;
            }
            if (ok && nblk > 0) {
                const CUtensorMap* kvm = a.kv_maps + b;
                const int plane_k = (a.layer * 2 + 0) * a.H + hh, plane_v = (a.layer * 2 + 1) * a.H + hh;
                mbar_expect_tx(q_full, 2 * AT_SUB);      // (its release also publishes s_off)
                tma_load_2d(&map_q, q_full, base + AT_OFF_Q, hh * AT_HD, off + row_base);
                tma_load_2d(&map_q, q_full, base + AT_OFF_Q + AT_SUB, hh * AT_HD + 64, off + row_base);
                // K stage j & 1 is free once the scores of block j - 2 are done, V stage once its P V is.
                auto load_k = [&](int j) -> bool {
                    if (j >= 2 && !at_wait(&k_empty[j & 1], (uint32_t)((j >> 1) - 1) & 1, s_flag)) return false;
                    uint8_t* dk = base + AT_OFF_K + (uint32_t)(j & 1) * 2 * AT_SUB;
                    const int key0 = (blk0 + j) * AT_BLK;
                    mbar_expect_tx(&k_full[j & 1], 2 * AT_SUB);
                    tma_load_3d(kvm, &k_full[j & 1], dk, 0, key0, plane_k);
                    tma_load_3d(kvm, &k_full[j & 1], dk + AT_SUB, 64, key0, plane_k);
                    return true;
                };
                auto load_v = [&](int j) -> bool {
                    if (j >= 2 && !at_wait(&v_empty[j & 1], (uint32_t)((j >> 1) - 1) & 1, s_flag)) return false;
                    uint8_t* dv = base + AT_OFF_V + (uint32_t)(j & 1) * 2 * AT_SUB;
                    const int key0 = (blk0 + j) * AT_BLK;
                    mbar_expect_tx(&v_full[j & 1], 2 * AT_SUB);
                    tma_load_3d(kvm, &v_full[j & 1], dv, 0, key0, plane_v);
                    tma_load_3d(kvm, &v_full[j & 1], dv + AT_SUB, 64, key0, plane_v);
                    return true;
                };
                // Requests follow the order in which the tensor core hands stages back
                // (S0 S1 PV0 S2 PV1 S3 ...): K0 V0 K1 V1 K2 K3 V2 K4 V3 K5 ...
                for (int j = n_pre; ok && j < 2 && j < nblk; ++j) ok = load_k(j) && load_v(j);
                for (int j = 2; ok && j < 4 && j < nblk; ++j) ok = load_k(j);
                for (int j = 2; ok && j < nblk; ++j) {
                    ok = load_v(j);
                    if (ok && j + 2 < nblk) ok = load_k(j + 2);
                }
            }
            if (!ok) { s_flag[0] = 1; atomicCAS(a.status, 0, (int)ADED_ERR_TIMEOUT); }
        }
    } else if (warp == 1) {
        // ---------------- MMA issuer (the whole warp runs this; one elected lane issues) ----------------
        if (nblk > 0) {
            // fp32 accumulate, bf16 operands; S: M 64 x N 64, both operands K-major; O: M 64 x N 128, B MN-major
            const uint32_t idesc_s = (1u << 4) | (1u << 7) | (1u << 10) | ((uint32_t)(64 >> 3) << 17) | ((uint32_t)(64 >> 4) << 24);
            const uint32_t idesc_o = (1u << 4) | (1u << 7) | (1u << 10) | (1u << 16) | ((uint32_t)(128 >> 3) << 17) | ((uint32_t)(64 >> 4) << 24);
            const uint64_t q_desc = smem_desc_sw128(smem_u32(base + AT_OFF_Q)), k_desc = smem_desc_sw128(smem_u32(base + AT_OFF_K));
            const uint64_t p_desc = smem_desc_sw128(smem_u32(base + AT_OFF_P)), v_desc = smem_desc_mn_sw128(smem_u32(base + AT_OFF_V), AT_SUB);
            bool ok = at_wait(q_full, 0, s_flag);
            __syncwarp();
            const uint32_t off0 = (uint32_t)s_off[0], off1 = (uint32_t)s_off[1];    // published by the producer before q
            // (Descriptor addresses are in 16-byte units.)
            auto issue_s = [&](int j) -> bool {
                const int s = j & 1;
                bool w = at_wait(&k_full[s], ((uint32_t)(j >> 1) + (s ? off1 : off0)) & 1, s_flag);
                if (j >= 2) w = w && at_wait(&s_empty[s], (uint32_t)((j >> 1) - 1) & 1, s_flag);
                if (!__all_sync(0xffffffffu, w)) return false;
                tc_fence_after();
                const uint64_t kd = k_desc + (uint64_t)((uint32_t)s * 2 * AT_SUB >> 4);
                const uint32_t d = tmem_base + AT_S_COL + (uint32_t)s * 64;
#pragma unroll
                for (int h = 0; h < 2; ++h) {
#pragma unroll
                    for (int kk = 0; kk < 4; ++kk)
                        tc_mma_bf16_elect(d, q_desc + (uint64_t)((h * AT_SUB + kk * 32) >> 4), kd + (uint64_t)((h * AT_SUB + kk * 32) >> 4), idesc_s,
                                          (h | kk) ? 1u : 0u);
                }
                tc_commit_elect(&k_empty[s]);
                tc_commit_elect(&s_full[s]);
                return true;
            };
            auto issue_pv = [&](int j) -> bool {
                const int s = j & 1;
                const bool w = at_wait(&p_full[s], (uint32_t)(j >> 1) & 1, s_flag) &&
                               at_wait(&v_full[s], ((uint32_t)(j >> 1) + (s ? off1 : off0)) & 1, s_flag);
                if (!__all_sync(0xffffffffu, w)) return false;
                tc_fence_after();
                const uint64_t pd = p_desc + (uint64_t)((uint32_t)s * AT_SUB >> 4), vd = v_desc + (uint64_t)((uint32_t)s * 2 * AT_SUB >> 4);
#pragma unroll
                for (int kk = 0; kk < 4; ++kk)
                    tc_mma_bf16_elect(tmem_base + AT_O_COL, pd + (uint64_t)((kk * 32) >> 4), vd + (uint64_t)((kk * 2048) >> 4), idesc_o, (j | kk) ? 1u : 0u);
                tc_commit_elect(&v_empty[s]);
                tc_commit_elect(&p_empty[s]);
                return true;
            };
            // Scores run two blocks ahead of the softmax (two S buffers), so a K stage is handed back early.
            ok = __all_sync(0xffffffffu, ok) && issue_s(0);
            if (ok && nblk > 1) ok = issue_s(1);
            for (int j = 0; ok && j < nblk; ++j) {
                ok = issue_pv(j);
                if (ok && j + 2 < nblk) ok = issue_s(j + 2);
            }
            if (!ok && lane == 0) { s_flag[0] = 1; atomicCAS(a.status, 0, (int)ADED_ERR_TIMEOUT); }
        }
    } else {
        // ---------------- softmax: warps 2..5, TMEM lane quarter = warp % 4 ----------------
        const int qt = warp & 3;
        const int row = qt * 16 + (lane & 15), half = lane >> 4;
        const int node = row_base + row;
        const bool valid = node < T;
        uint64_t mlo = 0, mhi = 0;
        if (valid && nblk > 0) { mlo = a.anc[2 * (off + node)]; mhi = a.anc[2 * (off + node) + 1]; }
        const uint32_t lane_addr = tmem_base + ((uint32_t)(qt * 32) << 16);
        float mrow = -INFINITY, lsum = 0.f;
        bool ok = true;
        for (int j = 0; j < nblk; ++j) {
            const int s = j & 1;
            if (!__all_sync(0xffffffffu, at_wait(&s_full[s], (uint32_t)(j >> 1) & 1, s_flag))) { ok = false; break; }
            tc_fence_after();
            uint32_t sr[32];
            tc_ld32_split<32>(lane_addr + AT_S_COL + (uint32_t)s * 64, sr);
            tc_fence_before();
            __syncwarp();
            if (lane == 0) mbar_arrive(&s_empty[s]);
            const int p0 = (blk0 + j) * AT_BLK + half * 32;     // cache position of this thread's first score
            if (p0 + 32 > L) {
#pragma unroll
                for (int c = 0; c < 32; ++c) {
                    const int jn = p0 + c - L;
                    bool keep = jn < 0;
                    if (!keep && jn < T) keep = jn < 64 ? (mlo >> jn) & 1 : (mhi >> (jn - 64)) & 1;
                    if (!keep) sr[c] = 0xff800000u;     // -inf
                }
            }
            float bm4[4] = {-INFINITY, -INFINITY, -INFINITY, -INFINITY};
#pragma unroll
            for (int c = 0; c < 32; ++c) bm4[c & 3] = fmaxf(bm4[c & 3], __uint_as_float(sr[c]));
            float bm = fmaxf(fmaxf(bm4[0], bm4[1]), fmaxf(bm4[2], bm4[3]));
            bm = fmaxf(bm, __shfl_xor_sync(0xffffffffu, bm, 16));
            // Integer reference (scores in the log2 domain), as in k_tree_attn_mma, but kept while a new
            // maximum exceeds it by at most AT_SLACK: numerators then reach 2^AT_SLACK instead of 1, which
            // changes nothing (scaling by a power of two commutes with the bf16 rounding and with the fp32
            // sums), and the costly rescaling of O in tensor memory becomes rare.
            const float cand = ceilf(bm * a.scale_log2);
            const float nm = mrow == -INFINITY ? cand : (cand > mrow + AT_SLACK ? cand : mrow);
            const float use = nm == -INFINITY ? 0.f : nm;
            const bool moved = mrow != nm && mrow != -INFINITY;
            if (__any_sync(0xffffffffu, moved)) {
                // Rare: rescale this thread's half row of O in place.  All P V products issued so far must
                // have completed (j > 0 here: a reference cannot move before the first block).
                const float corr = exp2f(mrow - use);
                if (!__all_sync(0xffffffffu, at_wait(&p_empty[(j - 1) & 1], (uint32_t)((j - 1) >> 1) & 1, s_flag))) { ok = false; break; }
                tc_fence_after();
#pragma unroll
                for (int part = 0; part < 2; ++part) {
                    uint32_t o[32];
                    tc_ld32_split<64>(lane_addr + AT_O_COL + (uint32_t)part * 32, o);
#pragma unroll
                    for (int c = 0; c < 32; ++c) o[c] = __float_as_uint(__uint_as_float(o[c]) * corr);
                    tc_st32_split<64>(lane_addr + AT_O_COL + (uint32_t)part * 32, o);
                }
                tc_fence_before();
                lsum *= corr;
            }
            mrow = nm;
            float ps4[4] = {0.f, 0.f, 0.f, 0.f};
            uint32_t pk[16];
#pragma unroll
            for (int c = 0; c < 32; c += 2) {
                const float e0 = at_ex2(fmaf(__uint_as_float(sr[c]), a.scale_log2, -use));
                const float e1 = at_ex2(fmaf(__uint_as_float(sr[c + 1]), a.scale_log2, -use));
                ps4[(c >> 1) & 3] += e0 + e1;
                pk[c >> 1] = at_pack(e0, e1);
            }
            lsum += (ps4[0] + ps4[1]) + (ps4[2] + ps4[3]);
            if (j >= 2 && !__all_sync(0xffffffffu, at_wait(&p_empty[s], (uint32_t)((j >> 1) - 1) & 1, s_flag))) { ok = false; break; }
            uint8_t* prow = base + AT_OFF_P + (uint32_t)s * AT_SUB + (uint32_t)row * 128;
#pragma unroll
            for (int cc = 0; cc < 4; ++cc) {
                const int chunk = half * 4 + cc;
                *reinterpret_cast<uint4*>(prow + ((chunk ^ (row & 7)) << 4)) = make_uint4(pk[4 * cc], pk[4 * cc + 1], pk[4 * cc + 2], pk[4 * cc + 3]);
            }
            asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
            __syncwarp();
            if (lane == 0) mbar_arrive(&p_full[s]);
        }
        // ---- park the unnormalised partial (O, reference, sum) for the cluster merge ----
        if (ok && nblk > 0) ok = __all_sync(0xffffffffu, at_wait(&p_empty[(nblk - 1) & 1], (uint32_t)((nblk - 1) >> 1) & 1, s_flag));
        if (!ok) { s_flag[0] = 1; atomicCAS(a.status, 0, (int)ADED_ERR_TIMEOUT); }
        float4* so4 = reinterpret_cast<float4*>(base + AT_OFF_SO);
        float* sml = reinterpret_cast<float*>(base + AT_OFF_SML);
        if (ok && nblk > 0) {
            tc_fence_after();
#pragma unroll
            for (int part = 0; part < 2; ++part) {
                uint32_t o[32];
                tc_ld32_split<64>(lane_addr + AT_O_COL + (uint32_t)part * 32, o);
#pragma unroll
                for (int c4 = 0; c4 < 8; ++c4) {
                    const int idx = half * 16 + part * 8 + c4;
                    so4[row * 32 + (idx ^ (row & 15))] = make_float4(__uint_as_float(o[4 * c4]), __uint_as_float(o[4 * c4 + 1]),
                                                                      __uint_as_float(o[4 * c4 + 2]), __uint_as_float(o[4 * c4 + 3]));
                }
            }
            tc_fence_before();
        } else {
            mrow = -INFINITY;
            lsum = 0.f;
#pragma unroll
            for (int c4 = 0; c4 < 16; ++c4) so4[row * 32 + ((half * 16 + c4) ^ (row & 15))] = make_float4(0.f, 0.f, 0.f, 0.f);
        }
        const float ltot = lsum + __shfl_xor_sync(0xffffffffu, lsum, 16);
        if (half == 0) { sml[row * 2] = mrow; sml[row * 2 + 1] = ltot; }
    }

    // ---- merge the splits of this (sequence, head, row block) across the cluster ----
    // CTA j combines rows j, j + S, ... from all S CTAs' shared memory:
    // out = sum_s O_s 2^(m_s - M) / sum_s l_s 2^(m_s - M), rounded to bf16.
    const int S = a.n_splits;
    if (S > 1) {
        asm volatile("barrier.cluster.arrive.release.aligned;" ::: "memory");
        asm volatile("barrier.cluster.wait.acquire.aligned;" ::: "memory");
    } else {
        __syncthreads();
    }
    const uint32_t so_addr = smem_u32(base + AT_OFF_SO), sml_addr = smem_u32(base + AT_OFF_SML);
    constexpr int QUADS = AT_HD / 4;
    const int t_here = pass_status == 0 ? min(max(T - row_base, 0), AT_ROWS) : 0;
    for (int item = threadIdx.x; item < ((t_here - split + S - 1) / S) * QUADS; item += AT_THREADS) {
        const int row = split + (item / QUADS) * S, q4 = item % QUADS;
        float ms[8], ls[8];
        float4 os[8];
#pragma unroll
        for (int s2 = 0; s2 < 8; ++s2) {
            ms[s2] = -INFINITY;
            ls[s2] = 0.f;
            os[s2] = make_float4(0.f, 0.f, 0.f, 0.f);
            if (s2 < S) {
                uint32_t rm, ro;
                asm volatile("mapa.shared::cluster.u32 %0, %1, %2;" : "=r"(rm) : "r"(sml_addr + (uint32_t)row * 8), "r"(s2));
                asm volatile("mapa.shared::cluster.u32 %0, %1, %2;" : "=r"(ro) : "r"(so_addr + (uint32_t)(row * 32 + (q4 ^ (row & 15))) * 16), "r"(s2));
                asm volatile("ld.shared::cluster.v2.f32 {%0, %1}, [%2];" : "=f"(ms[s2]), "=f"(ls[s2]) : "r"(rm));
                asm volatile("ld.shared::cluster.v4.f32 {%0, %1, %2, %3}, [%4];"
                             : "=f"(os[s2].x), "=f"(os[s2].y), "=f"(os[s2].z), "=f"(os[s2].w) : "r"(ro));
            }
        }
        float M = -INFINITY;
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
        bf16* dst = a.out + ((size_t)(off + row_base + row) * a.H + hh) * AT_HD + q4 * 4;
        uint2 u;
        u.x = at_pack(num.x * inv, num.y * inv);
        u.y = at_pack(num.z * inv, num.w * inv);
        *reinterpret_cast<uint2*>(dst) = u;
    }
    if (S > 1) {   // nobody may leave while a neighbour still reads its shared memory
        asm volatile("barrier.cluster.arrive.release.aligned;" ::: "memory");
        asm volatile("barrier.cluster.wait.acquire.aligned;" ::: "memory");
    }

    // ---------------- teardown ----------------
    tc_fence_before();
    __syncthreads();
    if (warp == 0 && lane == 0 && s_flag[0]) {
        // unwinding after a timeout: give copies that are still in flight time to land (bounded)
        for (int i = 0; i < 1000; ++i) __nanosleep(1000);
    }
    __syncthreads();
    if (warp == 1) {
        tc_fence_after();
        asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem_base), "r"((uint32_t)AT_TMEM_COLS) : "memory");
    }
}

// ---- host side --------------------------------------------------------------------------------
typedef CUresult (*AtEncodeFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*,
                               const cuuint64_t*, const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave,
                               CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

// Map over one sequence's cache block [planes][capacity][128] bf16 (planes = layers x {K, V} x heads):
// boxes of 64 positions x 64 elements, 128-byte swizzle, positions past the capacity read as zero.
bool attn_tc_make_kv_map(CUtensorMap* map, const void* block, uint64_t capacity, uint64_t planes) {
    static AtEncodeFn fn = nullptr;
    if (!fn) {
        void* p = nullptr;
        cudaDriverEntryPointQueryResult q;
        if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &p, cudaEnableDefault, &q) != cudaSuccess || q != cudaDriverEntryPointSuccess)
            return false;
        fn = reinterpret_cast<AtEncodeFn>(p);
    }
    const cuuint64_t dims[3] = {AT_HD, capacity, planes};
    const cuuint64_t strides[2] = {AT_HD * 2, capacity * AT_HD * 2};
    const cuuint32_t box[3] = {64, AT_BLK, 1};
    const cuuint32_t elem[3] = {1, 1, 1};
    return fn(map, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 3, const_cast<void*>(block), dims, strides, box, elem,
              CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
              CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

bool attn_tc_supported(const aded_model_config& c) { return c.dtype == ADED_BF16 && c.head_dim == AT_HD; }

// Raises the kernel's dynamic shared-memory limit; once per process, before any launch.
bool attn_tc_prepare() {
    return cudaFuncSetAttribute(k_tree_attn_tc, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)AT_SMEM) == cudaSuccess;
}

void launch_tree_attention_tc(aded_model* m, aded_kv* kv, int layer, int batch, int max_tree, cudaStream_t st) {
    AttnTcArgs a;
    a.kv_maps = kv->maps_dev;
    a.out = (bf16*)m->attn;
    a.len = kv->len_dev;
    a.row_off = m->seqs.row_off;
    a.anc = m->rows.anc;
    a.layer = layer;
    a.H = m->cfg.n_heads;
    // Trees of more than 64 nodes are two blocks of 64 query rows in separate CTAs.  Key splits per
    // (sequence, head, row block): up to 8 (one cluster), as many as keep the launch within the
    // two-per-SM CTA slots.
    a.row_blocks = max_tree <= AT_ROWS ? 1 : 2;
    int splits = ws_grid_limit(m->device) / (m->cfg.n_heads * batch * a.row_blocks);
    splits = splits < 1 ? 1 : splits > 8 ? 8 : splits;
    a.n_splits = splits;
    a.scale_log2 = 1.4426950408889634f / sqrtf((float)AT_HD);
    a.status = m->status;
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3(m->cfg.n_heads, splits, batch * a.row_blocks);
    cfg.blockDim = dim3(AT_THREADS);
    cfg.dynamicSmemBytes = AT_SMEM;
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
    cudaLaunchKernelEx(&cfg, k_tree_attn_tc, m->att_q_map, a);
}

}  // namespace aded
