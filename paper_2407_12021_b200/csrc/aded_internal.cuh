// Internal declarations shared by the library's translation units (not part of the ABI).
#pragma once

#include <cuda.h>
#include <cuda_bf16.h>
#include <cuda_runtime.h>
#include <stdint.h>

#include <vector>

#include "aded.h"
#include "gemm_out.cuh"

#define ADED_CUDA_TRY(expr)                      \
    do {                                         \
        cudaError_t _e = (expr);                 \
        if (_e != cudaSuccess) {                 \
            aded::note_cuda_error(_e, #expr);    \
            return ADED_ERR_CUDA;                \
        }                                        \
    } while (0)

namespace aded {

void note_cuda_error(cudaError_t e, const char* what);
void note_launch(int n = 1);   // bumps the process-wide launch counter

enum { ARGMAX_CHUNKS = 16 };
enum { PROF_GEMM = 0, PROF_ATTN = 1, PROF_OTHER = 2, PROF_GROUPS = 3 };
struct ProfSpan { int group; int launches; cudaEvent_t a, b; };

// ---- element types ---------------------------------------------------------------------
typedef __nv_bfloat16 bf16;

__device__ __forceinline__ float to_f32(float v) { return v; }
__device__ __forceinline__ float to_f32(bf16 v) { return __bfloat162float(v); }
template <typename T> __device__ __forceinline__ T from_f32(float v);
template <> __device__ __forceinline__ float from_f32<float>(float v) { return v; }
template <> __device__ __forceinline__ bf16 from_f32<bf16>(float v) { return __float2bfloat16_rn(v); }

// ---- programmatic dependent launch ---------------------------------------------------------
// Every kernel of a pass is launched with the programmatic-serialisation attribute and begins with
// pdl_enter(): it lets the next kernel of the stream start launching at once (its blocks become
// resident and run their own preamble) and then waits until the previous kernel has finished and
// its writes are visible.  Nothing may be read from or written to global memory that another kernel
// of the pass touches before pdl_wait() -- the weight-streaming GEMM alone does work before it: it
// prefetches weights, which no kernel writes.
__device__ __forceinline__ void pdl_launch_dependents() { asm volatile("griddepcontrol.launch_dependents;" ::: "memory"); }
__device__ __forceinline__ void pdl_wait() { asm volatile("griddepcontrol.wait;" ::: "memory"); }
__device__ __forceinline__ void pdl_enter() { pdl_launch_dependents(); pdl_wait(); }

// ---- index checks of the debug build -------------------------------------------------------------
// Compiled with -DADED_DEBUG_CHECKS (python -m paper_2407_12021_b200.build --debug -> libaded_debug.so) the
// kernels test the indices they are about to use on slots, cache rows and table buckets; a failed test
// records ADED_ERR_INTERNAL in the status word and the access is skipped.  In the product build the
// macro is the constant true and costs nothing.
#ifdef ADED_DEBUG_CHECKS
#define ADED_IN_RANGE(cond, status) ((cond) ? true : (atomicCAS(const_cast<int32_t*>(status), 0, (int)ADED_ERR_INTERNAL), false))
#else
#define ADED_IN_RANGE(cond, status) true
#endif

// ---- stage trace ---------------------------------------------------------------------------------
// The status word of a model is the first of a small block of device memory:
//   int32 [0] status, [1] trace switch, [2] marks taken, [3] unused; then TRACE_CAP 64-bit times (ns of
//   the global timer) and TRACE_CAP int32 kinds.
// While the switch is on, every kernel of a pass records, from one thread of its first block, the time at
// which its wait for the previous kernel ended.  The difference between two consecutive marks is the
// time the earlier kernel added to the pass (its overlap with its neighbours included), which is what
// a roofline report of a step chained by programmatic dependent launch needs; event pairs around
// launches would serialise the kernels.
enum { TRACE_CAP = 16384, STATUS_WORDS = 4 + 3 * TRACE_CAP };
enum { TK_OTHER = 0, TK_GEMM_QKV = 1, TK_GEMM_O = 2, TK_GEMM_GU = 3, TK_GEMM_DOWN = 4, TK_GEMM_HEAD = 5, TK_ATTN = 6,
       TK_NORM = 7, TK_ROPE = 8, TK_SWIGLU = 9, TK_PICK = 10, TK_STEP_END = 11 };
__device__ __forceinline__ void trace_mark(const int32_t* status, int kind) {
    int32_t* s = const_cast<int32_t*>(status);
    if (__ldcg(s + 1) == 0) return;
    const int i = atomicAdd(s + 2, 1) & (TRACE_CAP - 1);
    unsigned long long t;
    asm volatile("mov.u64 %0, %%globaltimer;" : "=l"(t));
    reinterpret_cast<unsigned long long*>(s + 4)[i] = t;
    (s + 4 + 2 * TRACE_CAP)[i] = kind;
}
__device__ __forceinline__ bool first_thread_of_grid() {
    return threadIdx.x == 0 && blockIdx.x == 0 && blockIdx.y == 0 && blockIdx.z == 0;
}

template <typename... KArgs, typename... Args>
inline cudaError_t launch_k(void (*kernel)(KArgs...), dim3 grid, dim3 block, size_t smem, cudaStream_t st, Args... args) {
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = grid;
    cfg.blockDim = block;
    cfg.dynamicSmemBytes = smem;
    cfg.stream = st;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr;
    cfg.numAttrs = 1;
    return cudaLaunchKernelEx(&cfg, kernel, KArgs(args)...);
}

// ---- per-call row bookkeeping (device arrays sized for max_rows / max_batch) --------------
struct RowMeta {
    int32_t* seq;      // [R] sequence of the row
    int32_t* local;    // [R] node index inside its tree
    int32_t* depth;    // [R] edges from the root
    int32_t* pos;      // [R] rotary position = committed length + depth
    uint64_t* anc;     // [R][2] bit j set <=> local node j is an ancestor of the row's node, or itself
};

// The caller's arrays of one verify/append call.  Kernels read them through this record, which
// lives at a fixed device address and is rewritten before every call, so that a captured launch
// sequence can be replayed with other arrays.
struct CallPtrs {
    const int32_t* tokens;
    const int32_t* parents;
    int32_t* out_tokens;
    int32_t* out_len;
    int32_t out_stride;
};

// Draft approval of one sequence, by one thread (a tree has at most ADED_MAX_NODES nodes; arrays in shared
// memory).  A node is approved when its parent is approved and its token equals the model's token at the
// parent; the deepest approved node (lowest index among equals) ends the accepted path.  Emits the
// model's token of every path node: the approved drafts' successors, ending with the model's own next
// token.  A failed pass emits nothing and keeps the committed length.
__device__ __forceinline__ void approval_walk(const int32_t* s_par, const int32_t* s_tok, const int32_t* s_best,
                                              const int32_t* s_dep, int T, int pass_status, int committed,
                                              int32_t* out_tokens, int32_t* out_len, int32_t* path, int32_t* new_len) {
    if (pass_status != 0) {
        *out_len = 0;
        *new_len = committed;
        return;
    }
    uint64_t ok_lo = 1ull, ok_hi = 0ull;   // approved set; the root always is
    int deepest = 0, deepest_depth = 0;
    for (int i = 1; i < T; ++i) {
        const int p = s_par[i];
        const bool p_ok = p < 64 ? (ok_lo >> p) & 1 : (ok_hi >> (p - 64)) & 1;
        if (p_ok && s_tok[i] == s_best[p]) {
            if (i < 64) ok_lo |= 1ull << i; else ok_hi |= 1ull << (i - 64);
            const int d = s_dep[i];
            if (d > deepest_depth) { deepest_depth = d; deepest = i; }
        }
    }
    // path[j] for j = depth .. 0 by climbing; the node at depth j is path element j
    int cur = deepest;
    for (int j = deepest_depth; j >= 0; --j) {
        path[j] = cur;
        out_tokens[j] = s_best[cur];
        cur = s_par[cur];
    }
    *out_len = deepest_depth + 1;
    *new_len = committed + deepest_depth + 1;
}

struct SeqMeta {
    int32_t* row_off;  // [B+1] first row of each sequence
    int32_t* path;     // [B][ADED_MAX_NODES] accepted path (local node indices), root first
    int32_t* new_len;  // [B] committed length after this call
};

}  // namespace aded

namespace aded {
// What the weight-streaming GEMM leaves behind (gemm_ws.cu): the partial tiles alone, or also -- the LM
// head -- per-row greedy candidates of every tile, reduced in the kernel's tail.
enum { WS_EPI_SLOTS = 0, WS_EPI_ARGMAX = 1 };
struct WsEpilogue {
    int mode;
    const TileRef* tiles;        // contributors of every tile
    uint32_t* counters;          // one arrival counter per tile; never reset: the epoch-th launch waits for
    uint32_t epoch;              //   n x epoch arrivals (modulo 2^32)
    float* cand_val; int32_t* cand_idx;   // best logit and its column per (row, tile): [R][n_tiles]
};
}  // namespace aded

struct aded_kv {
    const aded_model* model;
    int device;
    int batch;
    size_t elem;                  // bytes per element
    std::vector<int32_t> cap;     // host copy of capacities
    std::vector<char*> base;      // host copy of the per-sequence block pointers (device memory)
    char** base_dev;              // [B] device array of the same pointers
    int32_t* cap_dev;             // [B]
    int32_t* len_dev;             // [B] committed lengths
    CUtensorMap* maps_dev;        // [B] TMA descriptors of the blocks (tensor-core attention), or NULL
};

struct aded_model {
    aded_model_config cfg;
    int device;
    aded_weights top;
    std::vector<aded_layer_weights> layers;
    size_t elem;

    // activations, all [max_rows, *]
    void* h;        // residual stream            [R, d]   model dtype
    void* x;        // normalised input of a GEMM [R, d]
    void* q;        // rotated queries            [R, d]
    void* attn;     // attention output           [R, d]
    void* act;      // SwiGLU product             [R, F]
    float* y32;     // fp32 GEMM output, widest of 3d / 2F / d columns
    float* logits;  // [R, V] fp32
    float* rope_cos;  // [R, hd/2]
    float* rope_sin;
    int32_t* best;    // [R] greedy token per row
    int32_t* tokens;  // [R] staging for the _host entry points
    int32_t* parents;
    int32_t* out_tokens;   // [R]
    int32_t* out_len;      // [max_batch]
    int32_t* status;  // device status word
    aded::RowMeta rows;
    aded::SeqMeta seqs;
    aded::CallPtrs* call_dev;   // device copy of the current call's array pointers
    std::vector<void*> owned;   // everything cudaMalloc'ed for this handle

    // sampling-mode verification (aded_verify_sampled): armed for one call
    bool samp_on;
    float samp_temp, samp_top_p;
    const float* samp_u;        // caller's [rows] uniform numbers (device)

    void* step_mcts;            // scratch of aded_decode_step_mcts (allocated on first use)

    float* dbg_logits;
    int32_t* dbg_best;
    void* dbg_hidden;   // [n_layers + 1][rows][d] copies of the residual stream (debug capture)

    bool att_mma;       // bf16 models: tensor-core split-KV attention kernel
    bool att_tc;        // bf16 models with head_dim 128: the tcgen05 attention kernel (tree_attention_tc.cu)
    bool att_tc_ok;     // the tcgen05 kernel can be used (aded_debug_attention_kernel switches between the two)
    CUtensorMap att_q_map;   // TMA descriptor of q for it

    // tensor-core GEMM path (bf16 models): TMA descriptors and split-tile scratch
    bool ws_ready;
    std::vector<CUtensorMap> ws_maps;   // per layer: wqkv, wo, wgu, wd; then lm_head; then x, attn, act (boxes of 16 rows); then the same three with boxes of 64 rows
    std::vector<void*> ws_tiled;        // the weight matrices re-tiled for the tensor-core GEMM (same indices as ws_maps), model-owned
    bool ws_use_tiled;                  // GEMMs read the re-tiled copies (else the caller's matrices through ws_maps)
    float* ws_slots;                    // partial result tiles (see gemm_out.cuh)
    aded::TileRef* ws_tiles[5];         // contributor tables of the wqkv, wo, wgu, wd and LM-head results
    bool ws_one_per_sm[5];              // which of those five GEMMs launch one CTA per SM instead of two
    uint32_t* ws_counters;              // arrival counters of the LM head's tail, one per tile
    uint32_t ws_epoch;                  // LM-head launches with a tail so far (host side of the counters)
    float* cand_val;                    // [R][vocab / 128] per-tile greedy candidates of the LM head
    int32_t* cand_idx;

    float* norm_ssq;        // [R][32] per-chunk sums of squares of the RMSNorm kernel
    int32_t* norm_count;    // [R] chunk arrival counters, zero between launches
    float* argmax_val;      // [R][ARGMAX_CHUNKS] best logit of each column chunk
    int32_t* argmax_idx;

    bool prof_on;
    float prof_ms[aded::PROF_GROUPS];             // harvested so far
    int32_t prof_n[aded::PROF_GROUPS];
    std::vector<aded::ProfSpan> prof_spans;   // spans recorded by direct launches since aded_profile_begin
    std::vector<cudaEvent_t> prof_pool;       // events kept for reuse
};

namespace aded {

// ---- launchers (each enqueues on `st`; shapes are validated by the callers) ---------------
// tree.cu
void launch_tree_prologue(aded_model* m, aded_kv* kv, int batch, int chain_mode, cudaStream_t st);
void launch_accept(aded_model* m, aded_kv* kv, int batch, cudaStream_t st);
void launch_compact_commit(aded_model* m, aded_kv* kv, int batch, int chain_mode, cudaStream_t st);

// dense.cu
void launch_embed(aded_model* m, int rows, cudaStream_t st);
void launch_rope_table(aded_model* m, int rows, cudaStream_t st);
// `y` (may be NULL): projection result added to the residual stream before the norm
void launch_add_rmsnorm(aded_model* m, const GemmOut* y, const void* gain, int rows, cudaStream_t st);
// w_map / x_map: indices into m->ws_maps of the operands' TMA descriptors (-1: none, plain kernel).
// `y` is the fp32 buffer the plain kernel writes; the returned descriptor says where the result is.
// `epi_mode` (WS_EPI_*): whether the tensor-core kernel's tail also leaves per-tile greedy candidates (LM head).
GemmOut launch_gemm(aded_model* m, int w_map, int x_map, const void* x, const void* w, float* y, int rows, int n, int k,
                    int epi_mode, int trace_kind, cudaStream_t st);
void launch_rope_kv(aded_model* m, aded_kv* kv, const GemmOut& qkv, int layer, int rows, cudaStream_t st);
void launch_swiglu(aded_model* m, const GemmOut& gu, int rows, cudaStream_t st);
void launch_argmax(aded_model* m, const GemmOut& logits, int rows, cudaStream_t st);
// Writes a projection result as a plain [rows, n] fp32 matrix (debug paths).
void launch_materialize(aded_model* m, const GemmOut& src, float* dst, int rows, cudaStream_t st);

// dense_ws.cu: bf16 consumers of slot-resident projection results
void launch_add_rmsnorm_ws(aded_model* m, const GemmOut& y, const void* gain, int rows, cudaStream_t st);
void launch_swiglu_ws(aded_model* m, const GemmOut& gu, int rows, cudaStream_t st);
void launch_rope_kv_ws(aded_model* m, aded_kv* kv, const GemmOut& qkv, int layer, int rows, cudaStream_t st);
bool embed_norm_ws_supported(const aded_model* m);
// embedding lookup and the first RMSNorm in one kernel
void launch_embed_norm_ws(aded_model* m, const void* gain, int rows, cudaStream_t st);
// greedy token per row from the LM head's per-tile candidates, then the approval walk (one launch)
void launch_pick_accept(aded_model* m, aded_kv* kv, int batch, int n_tiles, cudaStream_t st);

// gemm_ws.cu
bool ws_make_map(CUtensorMap* map, const void* ptr, uint64_t rows, uint64_t cols, uint32_t box_rows);
bool ws_supported(int n, int k);
bool ws_prepare();
bool attn_prepare();
int ws_grid_limit(int device);
int ws_grid(int device, int n, int k, bool one_per_sm);
size_t ws_slot_floats(int device, int max_n, int max_rows);
cudaError_t ws_retile(const void* w, void* out, int n, int k, cudaStream_t st);
cudaError_t ws_launch(const CUtensorMap& map_w, const void* w_tiled, const CUtensorMap& map_x, const CUtensorMap& map_x64, int rows, int row0, int blk,
                      int n, int k,
                      float* slots, int32_t* status, const WsEpilogue& epi, int trace_kind, int device, bool one_per_sm, cudaStream_t st);
enum { WS_MAP_QKV = 0, WS_MAP_O = 1, WS_MAP_GU = 2, WS_MAP_D = 3 };   // per-layer map order
cudaError_t ws_wait_probe(int which, long long limit_cycles, const uint32_t* never_raised, int32_t* status, cudaStream_t st);

// sample.cu
bool sample_supported(int vocab);
cudaError_t launch_sample_rows(const float* logits, int rows, int vocab, int ld, float temperature, float top_p, const float* u,
                               int32_t* out, const int32_t* status, cudaStream_t st);

// tree_attention_tc.cu
bool attn_tc_supported(const aded_model_config& c);
bool attn_tc_prepare();
bool attn_tc_make_kv_map(CUtensorMap* map, const void* block, uint64_t capacity, uint64_t planes);
void launch_tree_attention_tc(aded_model* m, aded_kv* kv, int layer, int batch, int max_tree, cudaStream_t st);

// tree_attention.cu
// max_tree: most nodes any sequence's tree has in this call
void launch_tree_attention(aded_model* m, aded_kv* kv, int layer, int batch, int rows, int max_tree, cudaStream_t st);

}  // namespace aded
