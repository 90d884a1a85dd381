// Where a projection's fp32 result lives, and how its consumers read it.
//
// The plain GEMM writes y[r, n] directly.  The tensor-core weight-streaming GEMM splits its
// (W tile, k block) work units evenly over its CTAs, so a 128-column tile of the result is
// generally the sum of several CTAs' partial tiles.  Every CTA stores its partial tile to a slot, and
// whoever consumes the result -- the next kernel (rotary/K-V write, residual add + RMSNorm, SwiGLU,
// a captured logits matrix, sampling; dense_ws.cu, dense.cu) or, for the LM head's greedy candidates,
// the tail of the GEMM kernel itself (gemm_ws.cu) -- adds a tile's slots while it reads, always in
// ascending CTA order, so the sum is the same on every run.
//
// Slot numbering: the segment of tile t computed by CTA c goes to slot t + c.  Walking the units
// in order, (t, c) never decreases and one of them grows at every segment boundary, so the sums
// are distinct.  A slot holds [rb][128] floats (rb = rows of the pass padded to 16).  A pass takes up to 128
// rows, or up to 256 when the call has more than 128 (half as many passes over the weights); a call with more
// rows than one pass takes uses one slot region per pass.
#pragma once

#include <cuda_bf16.h>
#include <stdint.h>

namespace aded {

// The contributors of one tile: first slot and how many consecutive slots to add.
struct TileRef {
    int first_slot;
    int count;
};

struct GemmOut {
    const float* y;       // mode 0: [rows, n] row-major
    const float* slots;   // mode 1: partial tiles
    const TileRef* tiles; // mode 1: contributors of every tile (device table, one per GEMM shape)
    int mode;
    int n;                // result columns
    int n_tiles, kb, g;   // mode 1: 128-column tiles, k blocks per tile, CTAs of the GEMM launch
    int rows;             // rows of the whole result (all passes)
    int blk_shift;        // mode 1: log2 of the rows a pass takes (7 or 8)
};

// First work unit of CTA c when `units` units are split over `g` CTAs.
__host__ __device__ __forceinline__ long long ws_start(long long c, long long units, long long g) {
    return c * units / g;
}
// CTA that owns unit u.
__host__ __device__ __forceinline__ int ws_owner(long long u, long long units, long long g) {
    long long c = ((u + 1) * g - 1) / units;
    if (c >= g) c = g - 1;
    while (c > 0 && ws_start(c, units, g) > u) --c;
    while (c + 1 < g && ws_start(c + 1, units, g) <= u) ++c;
    return (int)c;
}

// Contributors of tile `tile` when n_tiles x kb units are split over g CTAs (host: fills the tables).
__host__ __device__ __forceinline__ TileRef gemm_tile_ref(int n_tiles, int kb, int g, int tile) {
    const long long units = (long long)n_tiles * kb;
    const int c_first = ws_owner((long long)tile * kb, units, g);
    const int c_last = ws_owner((long long)(tile + 1) * kb - 1, units, g);
    TileRef t;
    t.first_slot = tile + c_first;
    t.count = c_last - c_first + 1;
    return t;
}

// Rows padded to 16 of the pass that holds row r, and where that pass's slot region starts.
__device__ __forceinline__ int gemm_block_rb(const GemmOut& o, int r) {
    const int blk = 1 << o.blk_shift;
    const int left = o.rows - ((r >> o.blk_shift) << o.blk_shift);
    const int in_blk = left < blk ? left : blk;
    return (in_blk + 15) & ~15;
}
__device__ __forceinline__ const float* gemm_slot_row(const GemmOut& o, const TileRef& t, int r, int rb) {
    const size_t region = (size_t)(r >> o.blk_shift) * (size_t)(o.n_tiles + o.g) * ((size_t)128 << o.blk_shift);
    return o.slots + region + ((size_t)t.first_slot * rb + (r & ((1 << o.blk_shift) - 1))) * 128;
}

// Value of result element (r, tile * 128 + col) given the tile's contributors.
__device__ __forceinline__ float gemm_out_at(const GemmOut& o, const TileRef& t, int r, int col) {
    const int rb = gemm_block_rb(o, r);
    const float* p = gemm_slot_row(o, t, r, rb) + col;
    const size_t stride = (size_t)rb * 128;
    float sum = 0.f;
#pragma unroll 4
    for (int i = 0; i < t.count; ++i) sum += __ldcg(p + (size_t)i * stride);
    return sum;
}

// Any element, any mode.
__device__ __forceinline__ float gemm_out_load(const GemmOut& o, int r, int c) {
    if (o.mode == 0) return o.y[(size_t)r * o.n + c];
    return gemm_out_at(o, o.tiles[c >> 7], r, c & 127);
}

#ifdef __CUDACC__
__device__ __forceinline__ float4 f4_add(float4 a, float4 b) { return make_float4(a.x + b.x, a.y + b.y, a.z + b.z, a.w + b.w); }

// Columns col .. col+3 (col % 4 == 0) of tile t, row r: slots added in CTA order.
__device__ __forceinline__ float4 gemm_out_at4(const GemmOut& o, const TileRef& t, int r, int col) {
    const int rb = gemm_block_rb(o, r);
    const float* p = gemm_slot_row(o, t, r, rb) + col;
    const size_t stride = (size_t)rb * 128;
    float4 sum = make_float4(0.f, 0.f, 0.f, 0.f);
    // Up to GO_BATCH contributors are fetched at once (predicated loads, no branch between them) and
    // then added in CTA order: a projection with few tiles (O, down: 32 tiles over 296 CTAs) has about
    // ten contributors per tile, and a loop that fetched them four at a time cost three L2 round trips.
    constexpr int GO_BATCH = 12;
    for (int i0 = 0; i0 < t.count; i0 += GO_BATCH) {
        float4 v[GO_BATCH];
#pragma unroll
        for (int j = 0; j < GO_BATCH; ++j)
            v[j] = i0 + j < t.count ? __ldcg(reinterpret_cast<const float4*>(p + (size_t)(i0 + j) * stride)) : make_float4(0.f, 0.f, 0.f, 0.f);
#pragma unroll
        for (int j = 0; j < GO_BATCH; ++j)
            if (i0 + j < t.count) sum = f4_add(sum, v[j]);
    }
    return sum;
}

// The same gather in two steps, for kernels that need several tiles' values at once: first the loads of up
// to B contributors (predicated, no use of the values), then the sum in CTA order.  Issuing the loads of
// all gathers before the first sum puts them in flight together -- one L2 round trip instead of one per
// gather.  Only for tiles with at most B contributors: callers check t.count <= B and otherwise use
// gemm_out_at4.
template <int B>
__device__ __forceinline__ void gemm_out_fetch4(const GemmOut& o, const TileRef& t, int r, int col, float4 (&v)[B]) {
    const int rb = gemm_block_rb(o, r);
    const float* p = gemm_slot_row(o, t, r, rb) + col;
    const size_t stride = (size_t)rb * 128;
#pragma unroll
    for (int j = 0; j < B; ++j)
        v[j] = j < t.count ? __ldcg(reinterpret_cast<const float4*>(p + (size_t)j * stride)) : make_float4(0.f, 0.f, 0.f, 0.f);
}
template <int B>
__device__ __forceinline__ float4 gemm_out_sum4(const float4 (&v)[B], const TileRef& t) {
    float4 sum = make_float4(0.f, 0.f, 0.f, 0.f);
#pragma unroll
    for (int j = 0; j < B; ++j)
        if (j < t.count) sum = f4_add(sum, v[j]);
    return sum;
}

__device__ __forceinline__ uint2 pack4_bf16(float a, float b, float c, float d) {
    const __nv_bfloat162 lo = __floats2bfloat162_rn(a, b), hi = __floats2bfloat162_rn(c, d);
    uint2 u;
    u.x = *reinterpret_cast<const uint32_t*>(&lo);
    u.y = *reinterpret_cast<const uint32_t*>(&hi);
    return u;
}
__device__ __forceinline__ float4 unpack4_bf16(uint2 u) {
    const __nv_bfloat162 lo = *reinterpret_cast<const __nv_bfloat162*>(&u.x), hi = *reinterpret_cast<const __nv_bfloat162*>(&u.y);
    return make_float4(__low2float(lo), __high2float(lo), __low2float(hi), __high2float(hi));
}


// act = round(silu(gate) * up) for four adjacent columns.
__device__ __forceinline__ uint2 swiglu4(float4 g, float4 u) {
    return pack4_bf16(g.x / (1.f + expf(-g.x)) * u.x, g.y / (1.f + expf(-g.y)) * u.y,
                      g.z / (1.f + expf(-g.z)) * u.z, g.w / (1.f + expf(-g.w)) * u.w);
}

// Rotary embedding of four adjacent pairs (i .. i+3 with i+half .. i+half+3) of one head's q and k of
// row r, and the copy of v: gathers the QKV projection's partial tiles, rotates with the row's
// cos/sin, rounds to bf16 and (when `store`) writes q to qd and K/V to the cache rows kdst / vdst.
__device__ __forceinline__ void rope_kv_item(const GemmOut& qkv, const TileRef& tq, const TileRef& tk, const TileRef& tv, int r,
                                             int cq, int ck, int cv, int i, int half, const float* __restrict__ cs_row,
                                             const float* __restrict__ sn_row, __nv_bfloat16* qd, __nv_bfloat16* kdst,
                                             __nv_bfloat16* vdst, bool store) {
    float4 q0, q1, k0, k1, v0, v1;
    constexpr int RB = 6;      // the QKV projection's tiles have three to five contributors at the 7B and 13B widths
    if (tq.count <= RB && tk.count <= RB && tv.count <= RB) {
        float4 fq0[RB], fq1[RB], fk0[RB], fk1[RB], fv0[RB], fv1[RB];
        gemm_out_fetch4<RB>(qkv, tq, r, (cq + i) & 127, fq0);
        gemm_out_fetch4<RB>(qkv, tq, r, (cq + i + half) & 127, fq1);
        gemm_out_fetch4<RB>(qkv, tk, r, (ck + i) & 127, fk0);
        gemm_out_fetch4<RB>(qkv, tk, r, (ck + i + half) & 127, fk1);
        gemm_out_fetch4<RB>(qkv, tv, r, (cv + i) & 127, fv0);
        gemm_out_fetch4<RB>(qkv, tv, r, (cv + i + half) & 127, fv1);
        q0 = gemm_out_sum4<RB>(fq0, tq); q1 = gemm_out_sum4<RB>(fq1, tq);
        k0 = gemm_out_sum4<RB>(fk0, tk); k1 = gemm_out_sum4<RB>(fk1, tk);
        v0 = gemm_out_sum4<RB>(fv0, tv); v1 = gemm_out_sum4<RB>(fv1, tv);
    } else {
        q0 = gemm_out_at4(qkv, tq, r, (cq + i) & 127); q1 = gemm_out_at4(qkv, tq, r, (cq + i + half) & 127);
        k0 = gemm_out_at4(qkv, tk, r, (ck + i) & 127); k1 = gemm_out_at4(qkv, tk, r, (ck + i + half) & 127);
        v0 = gemm_out_at4(qkv, tv, r, (cv + i) & 127); v1 = gemm_out_at4(qkv, tv, r, (cv + i + half) & 127);
    }
    const float4 c = *reinterpret_cast<const float4*>(cs_row + i), s = *reinterpret_cast<const float4*>(sn_row + i);
    if (!store) return;
    *reinterpret_cast<uint2*>(qd + i) = pack4_bf16(q0.x * c.x - q1.x * s.x, q0.y * c.y - q1.y * s.y, q0.z * c.z - q1.z * s.z, q0.w * c.w - q1.w * s.w);
    *reinterpret_cast<uint2*>(qd + i + half) = pack4_bf16(q1.x * c.x + q0.x * s.x, q1.y * c.y + q0.y * s.y, q1.z * c.z + q0.z * s.z, q1.w * c.w + q0.w * s.w);
    *reinterpret_cast<uint2*>(kdst + i) = pack4_bf16(k0.x * c.x - k1.x * s.x, k0.y * c.y - k1.y * s.y, k0.z * c.z - k1.z * s.z, k0.w * c.w - k1.w * s.w);
    *reinterpret_cast<uint2*>(kdst + i + half) = pack4_bf16(k1.x * c.x + k0.x * s.x, k1.y * c.y + k0.y * s.y, k1.z * c.z + k0.z * s.z, k1.w * c.w + k0.w * s.w);
    *reinterpret_cast<uint2*>(vdst + i) = pack4_bf16(v0.x, v0.y, v0.z, v0.w);
    *reinterpret_cast<uint2*>(vdst + i + half) = pack4_bf16(v1.x, v1.y, v1.z, v1.w);
}
#endif

}  // namespace aded
