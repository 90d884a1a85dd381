// Sampling-mode token choice for the verification step ("Draft Construction and Verification": a
// token is sampled at every position and compared with the draft token; Figure 5 evaluates
// temperature and top-p).  The paper does not say how the token is drawn; the rule implemented here
// is exact integer arithmetic after one rounded exponential per logit, so that it can be checked bit
// for bit:
//   1. m = max logit; t = fl32(fl32(l - m) * c), c = fl32(log2(e) / temperature)
//   2. n = floor(t), f = t - n; r = P(f) (degree-6 polynomial for 2^f, Horner in float32 with
//      separately rounded multiplications and additions); weight q = floor(r * 2^30) >> (-n)
//   3. total = sum q; need = ceil(total * floor(top_p * 65536) / 65536)
//   4. nucleus = shortest prefix of the tokens ordered by (q descending, id ascending) whose weights
//      reach need; Z = its sum
//   5. target = floor(Z * floor(u * 2^24) / 2^24); the sample is the first nucleus token in id order
//      whose running nucleus sum exceeds target.
// One block of 1024 threads per row; a thread keeps the weights of its contiguous run of at most 32
// tokens in registers.  The nucleus comes from a three-pass radix selection on the weights (per-bin
// integer mass and count in shared memory), ties at the threshold enter in id order; the draw is a
// block-wide prefix sum in id order.  All sums are integers, so the result does not depend on the
// order of the atomic additions.
#include "aded_internal.cuh"

namespace aded {

constexpr int SM_THREADS = 1024, SM_PER = 32;

__device__ __forceinline__ unsigned long long warp_incl_scan_u64(unsigned long long v, int lane) {
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) {
        const unsigned long long t = __shfl_up_sync(0xffffffffu, v, o);
        if (lane >= o) v += t;
    }
    return v;
}

// Exclusive prefix sum over the block in thread order; *total receives the block sum.
__device__ __forceinline__ unsigned long long block_excl_scan_u64(unsigned long long v, unsigned long long* warp_sums,
                                                                  unsigned long long* total) {
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    const unsigned long long incl = warp_incl_scan_u64(v, lane);
    __syncthreads();                               // warp_sums may still be read from an earlier scan
    if (lane == 31) warp_sums[warp] = incl;
    __syncthreads();
    if (warp == 0) {
        const unsigned long long w = warp_sums[lane];
        const unsigned long long wi = warp_incl_scan_u64(w, lane);
        warp_sums[lane] = wi - w;                  // exclusive offsets of the warps
        if (lane == 31) warp_sums[32] = wi;
    }
    __syncthreads();
    *total = warp_sums[32];
    return warp_sums[warp] + incl - v;
}

__global__ void __launch_bounds__(SM_THREADS)
k_sample_rows(const float* __restrict__ logits, int vocab, int ld, float temperature, float top_p,
              const float* __restrict__ u, int32_t* __restrict__ out, const int32_t* status) {
    pdl_enter();
    if (status && first_thread_of_grid()) trace_mark(status, TK_PICK);
    if (status && *status != 0) return;
    __shared__ unsigned long long s_mass[2048];
    __shared__ unsigned int s_cnt[2048];
    __shared__ unsigned long long s_warp[33];
    __shared__ float s_max[32];
    __shared__ unsigned long long s_sel[3];        // selected bin, mass above it, (unused)
    const int row = blockIdx.x, tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const int per = (vocab + SM_THREADS - 1) / SM_THREADS;      // <= SM_PER
    const int v0 = tid * per;
    const float* lrow = logits + (size_t)row * ld;

    // 1. maximum (the logits are read again below rather than kept: 1024 threads leave 64 registers each)
    float mx = -INFINITY;
#pragma unroll
    for (int j = 0; j < SM_PER; ++j) {
        const int v = v0 + j;
        if (j < per && v < vocab) mx = fmaxf(mx, lrow[v]);
    }
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) mx = fmaxf(mx, __shfl_xor_sync(0xffffffffu, mx, o));
    if (lane == 0) s_max[warp] = mx;
    __syncthreads();
    mx = s_max[0];
#pragma unroll
    for (int i = 1; i < 32; ++i) mx = fmaxf(mx, s_max[i]);

    // 2. weights
    const float c = __fdiv_rn(1.4426950408889634f, temperature);
    unsigned int q[SM_PER];
    unsigned long long own = 0;
#pragma unroll
    for (int j = 0; j < SM_PER; ++j) {
        q[j] = 0;
        const int v = v0 + j;
        const float lv = (j < per && v < vocab) ? lrow[v] : -INFINITY;
        if (lv != -INFINITY) {                                    // a logit of -inf has weight 0
            const float t = __fmul_rn(__fsub_rn(lv, mx), c);
            const float n = floorf(t);
            const float f = __fsub_rn(t, n);
            float r = 0.00021795998327434063f;
            r = __fadd_rn(__fmul_rn(r, f), 0.0012414311058819294f);
            r = __fadd_rn(__fmul_rn(r, f), 0.009681269526481628f);
            r = __fadd_rn(__fmul_rn(r, f), 0.0554824136197567f);
            r = __fadd_rn(__fmul_rn(r, f), 0.24022991955280304f);
            r = __fadd_rn(__fmul_rn(r, f), 0.6931470036506653f);
            r = __fadd_rn(__fmul_rn(r, f), 1.0f);
            const unsigned int big = __float2uint_rz(__fmul_rn(r, 1073741824.f));
            const float sh = -n;                                  // >= 0, an integer
            q[j] = sh < 32.f ? big >> (unsigned int)sh : 0u;
            own += q[j];
        }
    }
    unsigned long long total;
    block_excl_scan_u64(own, s_warp, &total);

    // 3. mass the nucleus must reach
    const unsigned long long p16 = __float2uint_rd(__fmul_rn(top_p, 65536.f));
    const unsigned long long need = (total * p16 + 65535ull) >> 16;

    // 4. radix selection of the threshold weight: bits 30..20, 19..10, 9..0
    unsigned int prefix = 0, prefix_mask = 0;
    unsigned long long mass_above = 0;
    unsigned int cnt_eq = 0;
    const int shifts[3] = {20, 10, 0};
    const int widths[3] = {11, 10, 10};
#pragma unroll
    for (int pass = 0; pass < 3; ++pass) {
        const int sh = shifts[pass], bins = 1 << widths[pass];
        for (int i = tid; i < 2048; i += SM_THREADS) { s_mass[i] = 0; s_cnt[i] = 0; }
        __syncthreads();
#pragma unroll
        for (int j = 0; j < SM_PER; ++j) {
            if (q[j] != 0 && (q[j] & prefix_mask) == prefix) {
                const unsigned int b = (q[j] >> sh) & (bins - 1);
                atomicAdd(&s_mass[b], (unsigned long long)q[j]);
                atomicAdd(&s_cnt[b], 1u);
            }
        }
        __syncthreads();
        // thread t owns bins 2047 - 2t and 2046 - 2t (descending), so that an exclusive scan in thread
        // order gives the mass of all higher bins
        const int b_hi = 2047 - 2 * tid, b_lo = 2046 - 2 * tid;
        const unsigned long long m_hi = b_hi < bins ? s_mass[b_hi] : 0ull, m_lo = b_lo < bins ? s_mass[b_lo] : 0ull;
        unsigned long long dummy;
        const unsigned long long above = block_excl_scan_u64(m_hi + m_lo, s_warp, &dummy);
        const unsigned long long rem = need - mass_above;          // still to be found among the candidates
        if (m_hi != 0 && above < rem && rem <= above + m_hi) { s_sel[0] = (unsigned long long)b_hi; s_sel[1] = above; }
        if (m_lo != 0 && above + m_hi < rem && rem <= above + m_hi + m_lo) { s_sel[0] = (unsigned long long)b_lo; s_sel[1] = above + m_hi; }
        __syncthreads();
        const unsigned int sel = (unsigned int)s_sel[0];
        mass_above += s_sel[1];
        cnt_eq = s_cnt[sel];
        prefix |= sel << sh;
        prefix_mask |= (unsigned int)(bins - 1) << sh;
        __syncthreads();
    }
    const unsigned int thr = prefix;                               // the smallest weight inside the nucleus
    const unsigned long long rem = need - mass_above;
    const unsigned long long n_ties = (rem + thr - 1) / thr;       // of the cnt_eq tokens with weight thr, lowest ids first
    const unsigned long long z = mass_above + n_ties * thr;
    (void)cnt_eq;

    // 5. rank the ties in id order, then draw in id order
    unsigned long long my_ties = 0;
#pragma unroll
    for (int j = 0; j < SM_PER; ++j) my_ties += q[j] == thr;
    unsigned long long dummy;
    unsigned long long tie_rank = block_excl_scan_u64(my_ties, s_warp, &dummy);
    unsigned long long my_mass = 0;
    unsigned int member = 0;                                       // bit j: token v0 + j is in the nucleus
#pragma unroll
    for (int j = 0; j < SM_PER; ++j) {
        bool in = q[j] > thr;
        if (q[j] == thr) { in = tie_rank < n_ties; ++tie_rank; }
        if (in) { member |= 1u << j; my_mass += q[j]; }
    }
    const unsigned long long before = block_excl_scan_u64(my_mass, s_warp, &dummy);
    unsigned long long u24 = __float2uint_rd(__fmul_rn(u[row], 16777216.f));
    if (u24 > 16777215ull) u24 = 16777215ull;                      // u must lie in [0, 1); anything else draws the last token
    const unsigned long long target = (__umul64hi(z, u24) << 40) | ((z * u24) >> 24);
    if (before <= target && target < before + my_mass) {
        unsigned long long run = before;
#pragma unroll
        for (int j = 0; j < SM_PER; ++j) {
            if (member & (1u << j)) {
                run += q[j];
                if (run > target) { out[row] = v0 + j; break; }
            }
        }
    }
}

bool sample_supported(int vocab) { return vocab >= 1 && vocab <= SM_THREADS * SM_PER; }

cudaError_t launch_sample_rows(const float* logits, int rows, int vocab, int ld, float temperature, float top_p, const float* u,
                               int32_t* out, const int32_t* status, cudaStream_t st) {
    return launch_k(k_sample_rows, dim3(rows), dim3(SM_THREADS), 0, st, logits, vocab, ld, temperature, top_p, u, out, status);
}

}  // namespace aded

using namespace aded;

extern "C" aded_status aded_sample_tokens(const float* logits_dev, int32_t rows, int32_t vocab, float temperature, float top_p,
                                          const float* u_dev, int32_t* out_tokens_dev, void* stream) {
    if (!logits_dev || !u_dev || !out_tokens_dev || rows < 1) return ADED_ERR_INVALID_ARG;
    if (!(temperature > 0.f) || !(top_p >= 1.f / 65536.f) || !(top_p <= 1.f)) return ADED_ERR_INVALID_ARG;
    if (!sample_supported(vocab)) return ADED_ERR_UNSUPPORTED;
    note_launch();
    ADED_CUDA_TRY(launch_sample_rows(logits_dev, rows, vocab, vocab, temperature, top_p, u_dev, out_tokens_dev, nullptr,
                                     static_cast<cudaStream_t>(stream)));
    return ADED_OK;
}
