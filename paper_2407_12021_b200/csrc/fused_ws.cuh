// Parameters of the persistent projection kernel (fused_ws.cu).
#pragma once

#include <cuda.h>
#include <cuda_bf16.h>
#include <stdint.h>

#include "gemm_out.cuh"

namespace aded {

constexpr int FW_MAX_PAIRS = 4;
constexpr int FW_COUNTERS = 64;        // launches per pass that get barrier counters (a pair each)

enum { FW_POST_NONE = 0, FW_POST_ADD_NORM = 1, FW_POST_SWIGLU = 2, FW_POST_ROPE_KV = 3 };

// One projection and the step that consumes its result.
struct FwPair {
    int map_w, map_x;          // indices into the device array of TMA descriptors
    int n_tiles, kb;           // W is [128 * n_tiles, 64 * kb]
    const TileRef* tiles;      // contributor table of the result
    int post;                  // FW_POST_*
    int layer;                 // FW_POST_ROPE_KV: layer whose K/V rows are written
    const void* gain;          // FW_POST_ADD_NORM: RMSNorm gain [d]
};

struct FwParams {
    int n_pairs;
    FwPair pair[FW_MAX_PAIRS];
    int rows, rb, stages, tmem_cols;
    const CUtensorMap* maps;
    float* slots;
    uint32_t* counter;         // this launch's two barrier counters (projections done, steps done), zero at launch
    int32_t* status;
    __nv_bfloat16 *h, *x, *q, *act;
    int d, F, H, hd;
    float eps;
    const float *rope_cos, *rope_sin;
    char* const* kv_base;
    const int32_t *kv_cap, *kv_len, *row_seq, *row_local;
};

}  // namespace aded
