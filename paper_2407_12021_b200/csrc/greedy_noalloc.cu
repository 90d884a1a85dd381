// aded_greedy_noalloc: the per-row greedy choice (largest fp32 logit, lowest token id among equals)
// over a logits matrix the caller already holds, for callers that must not allocate device memory.
//
// Who needs this: a serving process in which another component owns the whole device heap (a
// framework's caching allocator has reserved it, so a cudaMalloc from this library could fail or
// stall the device), or a latency-critical decode loop that forbids allocation calls altogether
// because cudaMalloc/cudaFree synchronise the device.  Such a caller cannot create a model handle
// (that allocates the activation workspace) but can still run the library's token choice on logits
// produced elsewhere.
//
// The two-stage reduction keeps its per-chunk partial results in a fixed file-scope device array
// instead of a workspace: 128 rows x 16 chunks x 8 bytes = 16 KiB, held by every device that loads
// the library until the process exits.  All calls share that array; see the header for the rules.
#include <mutex>

#include "aded_internal.cuh"

namespace aded {

constexpr int NA_MAX_ROWS = ADED_NOALLOC_MAX_ROWS;
constexpr int NA_CHUNKS = 16;

struct NaPartial { float value; int32_t index; };

// The scratch.  In host code this name is only a handle for cudaGetSymbolAddress -- it is not a
// device address and must never be passed to a kernel; device code could name it directly.
static __device__ __align__(256) NaPartial g_na_scratch[NA_MAX_ROWS * NA_CHUNKS];

// Stage 1: grid (chunks, rows); each block scans its column chunk of one row and leaves the best
// (value, index) in the scratch entry [row][chunk].  Every entry stage 2 reads is written here first,
// so nothing needs clearing between calls.
__global__ void __launch_bounds__(256) k_na_chunks(const float* __restrict__ logits, NaPartial* __restrict__ scratch,
                                                   int vocab, int chunk) {
    __shared__ float sv[8];
    __shared__ int si[8];
    const int r = blockIdx.y;
    const long long c0 = (long long)blockIdx.x * chunk;
    const long long c1 = c0 + chunk < vocab ? c0 + chunk : vocab;
    const float* row = logits + (size_t)r * vocab;
    float bv = -INFINITY;
    int bi = 0x7fffffff;
    for (long long c = c0 + threadIdx.x; c < c1; c += 256) {
        const float v = row[c];
        if (v > bv) { bv = v; bi = (int)c; }   // c ascends per thread: the first maximum is kept
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
        scratch[r * NA_CHUNKS + blockIdx.x].value = bv;
        scratch[r * NA_CHUNKS + blockIdx.x].index = bi;
    }
}

// Stage 2: one thread per row takes the best of the row's chunks (the lowest index wins among
// equal values).
__global__ void k_na_final(const NaPartial* __restrict__ scratch, int32_t* __restrict__ best, int rows) {
    const int r = blockIdx.x * blockDim.x + threadIdx.x;
    if (r >= rows) return;
    float bv = -INFINITY;
    int bi = 0x7fffffff;
    for (int i = 0; i < NA_CHUNKS; ++i) {
        const NaPartial p = scratch[r * NA_CHUNKS + i];
        if (p.value > bv || (p.value == bv && p.index < bi)) { bv = p.value; bi = p.index; }
    }
    best[r] = bi == 0x7fffffff ? 0 : bi;
}

// Device address of the scratch array, resolved once per device with that device current.
static aded_status na_scratch_address(NaPartial** out) {
    static std::mutex mu;
    static NaPartial* addr[64] = {};
    int dev = 0;
    ADED_CUDA_TRY(cudaGetDevice(&dev));
    if (dev < 0 || dev >= 64) return ADED_ERR_UNSUPPORTED;
    std::lock_guard<std::mutex> lock(mu);
    if (addr[dev] == nullptr) {
        void* p = nullptr;
        ADED_CUDA_TRY(cudaGetSymbolAddress(&p, g_na_scratch));
        addr[dev] = static_cast<NaPartial*>(p);
    }
    *out = addr[dev];
    return ADED_OK;
}

}  // namespace aded

using namespace aded;

extern "C" aded_status aded_greedy_noalloc(const float* logits_dev, int32_t rows, int32_t vocab, int32_t* out_best_dev,
                                          void* stream) {
    if (!logits_dev || !out_best_dev || rows < 1 || vocab < 1) return ADED_ERR_INVALID_ARG;
    if (rows > NA_MAX_ROWS) return ADED_ERR_INVALID_ARG;   // beyond the fixed scratch array
    NaPartial* scratch = nullptr;
    const aded_status s = na_scratch_address(&scratch);
    if (s != ADED_OK) return s;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    const int chunk = (int)(((long long)vocab + NA_CHUNKS - 1) / NA_CHUNKS);      // (64-bit: vocab may be close to INT_MAX)
    k_na_chunks<<<dim3(NA_CHUNKS, rows), 256, 0, st>>>(logits_dev, scratch, vocab, chunk);
    k_na_final<<<(rows + 127) / 128, 128, 0, st>>>(scratch, out_best_dev, rows);
    ADED_CUDA_TRY(cudaGetLastError());
    note_launch(2);
    return ADED_OK;
}
