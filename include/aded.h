/*
 * aded.h -- C ABI of the B200 verification-step library for adaptive draft-verification
 * decoding (ADED, "Adaptive Draft-Verification for Efficient Large Language Model Decoding").
 *
 * The library implements, for one GPU, the target-model side of the paper's loop
 * (Methodology, Fig. 2): score a whole draft token tree in one forward pass with tree
 * attention, approve drafts greedily, keep the approved path in the KV cache
 * ("Draft Construction and Verification"); raise the tri-gram counts of freshly produced
 * tokens (Algorithm 2); and list the most probable continuations of a two-token context
 * (Eq. 1; "get potential words from tri-gram matrix", Algorithm 1).
 *
 * Conventions
 *  - Every function returns an aded_status.  No exceptions, no global state.  A handle must
 *    not be used from two threads at once; distinct handles are independent.
 *  - Pointers named *_dev are DEVICE pointers on the device that was current when the handle
 *    was created; pointers named *_host are HOST pointers.  The caller owns both and keeps
 *    them alive until the work has finished on the stream.
 *  - `stream` is a cudaStream_t passed as void* (NULL = the legacy default stream).  Calls
 *    taking device pointers only enqueue work and never synchronise -- except those whose
 *    comment says "synchronises" (aded_kv_len, aded_kv_load, aded_kv_set_len, the poll_status
 *    calls, aded_trigram_get/stats/export/prune/save/load, aded_profile_end, aded_trace_begin/end):
 *    they hand a host value to or from the device and return after the stream has drained.
 *    Calls with a _host suffix copy their arguments in and their results out and likewise
 *    return after the stream has drained.
 *  - Device memory: handles allocate their workspace, cache blocks and tables with cudaMalloc
 *    when they are created (and aded_trigram_prune / aded_decode_step_mcts once more on first
 *    use) and free it when they are destroyed; the weights stay the caller's.  Nothing is
 *    allocated by the calls of a decoding step.
 *  - Errors the host can see (NULL handles, sizes out of range) are returned at once and
 *    nothing is launched.  Errors only the device can see (malformed parent array, cache
 *    capacity, hash table full, a bounded wait that ran out) are recorded in a device status
 *    word: the offending call leaves the cache/table unchanged and reports accept length 0,
 *    later calls on the handle do nothing until the handle's poll_status call has read and
 *    cleared it.
 */
#ifndef ADED_H
#define ADED_H

#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef enum aded_status {
    ADED_OK = 0,
    ADED_ERR_INVALID_ARG = 1,
    ADED_ERR_BAD_TREE = 2,     /* parents[0] != -1, or parents[i] not in [0, i) */
    ADED_ERR_KV_CAPACITY = 3,  /* committed length + tree nodes exceeds the sequence's capacity */
    ADED_ERR_TABLE_FULL = 4,   /* tri-gram store out of buckets */
    ADED_ERR_OOM = 5,
    ADED_ERR_CUDA = 6,
    ADED_ERR_UNSUPPORTED = 7,
    ADED_ERR_TIMEOUT = 8,      /* a bounded device-side wait ran out */
    ADED_ERR_INTERNAL = 9      /* debug build only: an index check inside a kernel failed (the access was skipped) */
} aded_status;

enum { ADED_F32 = 0, ADED_BF16 = 1 };

/* Most nodes (root included) one sequence's draft tree may have. */
#define ADED_MAX_NODES 128

/* Llama-style decoder widths.  head_dim must be 64 or 128, d_model = n_heads * head_dim.
 * dtype is the storage type of weights, activations and the KV cache; accumulation is fp32. */
typedef struct aded_model_config {
    int32_t n_layers, d_model, n_heads, head_dim, d_ffn, vocab;
    int32_t dtype;          /* ADED_F32 or ADED_BF16 */
    float rms_eps;          /* RMSNorm epsilon */
    float rope_theta;       /* rotary base */
    int32_t max_rows;       /* most tree nodes summed over the batch in one verify call (>= 1) */
    int32_t max_batch;      /* most sequences in one verify call (>= 1) */
} aded_model_config;

/* Device pointers to row-major weights, output feature major ([out, in]); BORROWED: they must
 * outlive the model.  (bf16 models also keep a re-tiled private copy of the matrices, made in
 * aded_model_create: see aded_debug_weight_layout.  Changing the caller's matrices afterwards is
 * not supported.)  wqkv [3d, d] holds the query rows, then key rows, then value rows, head h
 * owning rows h*head_dim .. (h+1)*head_dim - 1 of each block; wgu [2F, d] holds the gate rows
 * then the up rows; rotary pairs are (i, i + head_dim/2) within a head. */
typedef struct aded_layer_weights {
    const void *wqkv, *wo, *wgu, *wd, *norm1, *norm2;
} aded_layer_weights;

typedef struct aded_weights {
    const void* embed;                 /* [vocab, d] */
    const void* final_norm;            /* [d] */
    const void* lm_head;               /* [vocab, d] */
    const aded_layer_weights* layers;  /* HOST array of n_layers entries (copied) */
} aded_weights;

typedef struct aded_trigram_config {
    int32_t vocab;            /* token ids are 0 .. vocab-1 */
    int32_t log2_buckets;     /* 2^log2_buckets home buckets (one per two-token context), 4..28 */
    int32_t overflow_buckets; /* extra buckets for contexts with more than 6 continuations */
    uint32_t cap;             /* counts saturate here (Algorithm 2's maximum); 0 = 2^31 - 1, which is also the largest allowed */
    uint32_t min_count;       /* top-k skips entries below this count; 0 = off */
} aded_trigram_config;

typedef struct aded_model aded_model;     /* opaque, owned by the library */
typedef struct aded_kv aded_kv;
typedef struct aded_trigram aded_trigram;

/* ---- lifetime ------------------------------------------------------------------------- */

/* Validates the configuration, copies the weight pointer table and allocates the activation
 * workspace for max_rows rows.  ADED_ERR_UNSUPPORTED for widths the kernels do not cover,
 * ADED_ERR_OOM / ADED_ERR_CUDA if the device refuses. */
aded_status aded_model_create(const aded_model_config* cfg, const aded_weights* weights, aded_model** out);
aded_status aded_model_destroy(aded_model* m);

/* KV cache for `batch` sequences (<= the model's max_batch); capacity_host[b] positions for
 * sequence b.  Per sequence the cache is one block laid out
 * [layer][K|V][head][position][head_dim] in the model dtype.  All committed lengths start at 0
 * and live on the device. */
aded_status aded_kv_create(const aded_model* m, int32_t batch, const int32_t* capacity_host, aded_kv** out);
aded_status aded_kv_destroy(aded_kv* kv);
/* Committed length of sequence `seq`; synchronises `stream`. */
aded_status aded_kv_len(const aded_kv* kv, int32_t seq, int32_t* out_len_host, void* stream);
/* Overwrite positions [0, n_pos) of layer `layer` of sequence `seq` with given keys/values
 * (device pointers, [head][n_pos][head_dim], model dtype) and set the committed length to
 * n_pos.  For workloads that start from a pre-filled cache.  Synchronises `stream`. */
aded_status aded_kv_load(aded_kv* kv, int32_t seq, int32_t layer, const void* k_dev, const void* v_dev,
                         int32_t n_pos, void* stream);
/* Set the committed length of sequence `seq` to new_len (0 <= new_len <= capacity): roll a
 * sequence back to an earlier point, e.g. to the end of its prompt.  Rows past new_len stay in
 * memory and are overwritten by later calls.  Synchronises `stream`. */
aded_status aded_kv_set_len(aded_kv* kv, int32_t seq, int32_t new_len, void* stream);
/* Copy out positions [pos0, pos0 + n_pos) of one layer: k_dev / v_dev receive
 * [head][n_pos][head_dim].  For tests. */
aded_status aded_kv_read(const aded_kv* kv, int32_t seq, int32_t layer, int32_t pos0, int32_t n_pos,
                         void* k_dev, void* v_dev, void* stream);

/* Put n committed tokens (1 <= n <= min(max_rows, 128)) into the cache of sequence `seq`:
 * the verification pipeline on a chain whose every node is accepted, without the LM head. */
aded_status aded_append(aded_model* m, aded_kv* kv, int32_t seq, const int32_t* tokens_dev, int32_t n,
                        void* stream);

/* ---- the verification step ("Draft Construction and Verification") ---------------------- */

/* Verify one draft tree against the model for the single sequence of `kv` (batch 1).
 *   tree_tokens_dev[n_nodes]  token of each node; node 0 is the last committed token, whose
 *                             K/V are not cached yet (last prompt token or previous bonus token)
 *   tree_parents_dev[n_nodes] parent index, -1 for node 0, otherwise in [0, i)
 *   out_tokens_dev[n_nodes]   receives the emitted tokens: the model's greedy token after the
 *                             root, then after each approved draft; entries past accept_len
 *                             are left alone
 *   out_accept_len_dev[1]     approved drafts + 1 (the model's own token always counts);
 *                             0 if the call failed on the device
 * Each node attends to all committed positions and to its ancestors and itself; rotary
 * position = committed length + depth.  Greedy choice = largest fp32 logit, lowest id among
 * equals.  Approval walks from the root to the child whose token equals the parent's greedy
 * token until none matches.  Afterwards the K/V of the approved nodes sit at positions
 * L .. L+accept_len-1 and the committed length is L + accept_len. */
aded_status aded_verify(aded_model* m, aded_kv* kv, const int32_t* tree_tokens_dev,
                        const int32_t* tree_parents_dev, int32_t n_nodes, int32_t* out_tokens_dev,
                        int32_t* out_accept_len_dev, void* stream);

/* Same for every sequence of `kv` at once.  tree_offsets_host[batch + 1] gives each sequence's
 * slice of the concatenated token/parent arrays (parents are local to the slice; each slice has
 * 1..ADED_MAX_NODES nodes; the total is at most max_rows).  Sequence b's emitted tokens go to
 * out_tokens_dev[b * out_stride ...] (out_stride >= its node count). */
aded_status aded_verify_batch(aded_model* m, aded_kv* kv, const int32_t* tree_offsets_host,
                              const int32_t* tree_tokens_dev, const int32_t* tree_parents_dev,
                              int32_t* out_tokens_dev, int32_t out_stride, int32_t* out_accept_len_dev,
                              void* stream);

/* aded_verify with HOST arrays: copies the tree in, runs, copies the results out, waits. */
aded_status aded_verify_host(aded_model* m, aded_kv* kv, const int32_t* tree_tokens_host,
                             const int32_t* tree_parents_host, int32_t n_nodes, int32_t* out_tokens_host,
                             int32_t* out_accept_len_host, void* stream);

/* Sampling-mode verification ("Draft Construction and Verification": at every position a token is
 * sampled from the model's distribution and compared with the draft token; Figure 5: temperature and
 * top-p).  Same as aded_verify, except that node i's token is drawn with the uniform number u_dev[i]
 * (float32 in [0, 1), device, n_nodes of them, supplied by the caller -- the library draws no random
 * numbers) from softmax(logits / temperature) restricted to the top-p nucleus, by the rule of
 * aded_sample_tokens.  temperature > 0, 2^-16 <= top_p <= 1, vocab <= 32768, else
 * ADED_ERR_INVALID_ARG / ADED_ERR_UNSUPPORTED. */
aded_status aded_verify_sampled(aded_model* m, aded_kv* kv, const int32_t* tree_tokens_dev,
                                const int32_t* tree_parents_dev, int32_t n_nodes, float temperature, float top_p,
                                const float* u_dev, int32_t* out_tokens_dev, int32_t* out_accept_len_dev, void* stream);

/* The drawing rule alone: out_tokens_dev[r] for r < rows from logits_dev[r][0 .. vocab) (float32, row
 * stride vocab, finite or -inf) and u_dev[r].  The paper does not fix a rule; this one is exact
 * integer arithmetic after one rounded exponential per logit, so two implementations agree bit for
 * bit:  m = max logit;  t = fl32(fl32(l - m) * fl32(log2(e) / temperature));  n = floor(t), f = t - n;
 * r = 2^f by a fixed degree-6 polynomial in float32 (Horner, every product and sum rounded);
 * weight q = floor(r * 2^30) >> (-n);  need = ceil(sum q * floor(top_p * 65536) / 65536);  nucleus =
 * shortest prefix in (q descending, id ascending) order with mass >= need, Z its mass;  target =
 * floor(Z * floor(u * 2^24) / 2^24);  result = first nucleus token in id order whose running mass
 * exceeds target.  Asynchronous on `stream`. */
aded_status aded_sample_tokens(const float* logits_dev, int32_t rows, int32_t vocab, float temperature, float top_p,
                               const float* u_dev, int32_t* out_tokens_dev, void* stream);

/* Ask the next verify call to also write every node's logits ([rows][vocab] fp32, may be NULL)
 * and greedy token ([rows] int32, may be NULL) to the given device buffers.  Parity checks only. */
aded_status aded_debug_capture(aded_model* m, float* logits_dev, int32_t* best_dev);

/* Run one of the model's projections alone, through the same kernel the verification step uses:
 * y[rows, N] (fp32) = x[rows, K] (model dtype) * W^T, with W = layer `layer`'s wqkv (which = 0),
 * wo (1), wgu (2), wd (3), or the LM head (4; layer ignored).  rows <= max_rows.  Parity checks of
 * the dense contraction ("forward pass through the model", Introduction) only. */
aded_status aded_debug_gemm(aded_model* m, int32_t layer, int32_t which, const void* x_dev, int32_t rows,
                            float* y_dev, void* stream);

/* Per-kernel timing for roofline reports (not part of the paper's method).  Between begin and end
 * every launch of the model's kernels is bracketed by CUDA events on its stream, grouped as
 * 0 = projection/FFN/LM-head GEMMs, 1 = tree attention, 2 = everything else.  end() synchronises
 * the stream and writes the summed milliseconds and launch counts of each group (arrays of 3). */
aded_status aded_profile_begin(aded_model* m);
aded_status aded_profile_end(aded_model* m, float* out_ms_host, int32_t* out_launches_host, void* stream);
/* Kernels launched by this library in this process so far (all handles). */
uint64_t aded_launch_count(void);

/* Stage trace of the verification step as it really runs, kernels overlapping under programmatic
 * dependent launch (not part of the paper's method; the per-launch events of aded_profile_begin serialise
 * the kernels, this does not).  Between begin and end every kernel of a pass records, from one thread,
 * the device's global-timer value (ns) at the moment its wait for the previous kernel ended, with a
 * kind: 0 other, 1..5 the QKV / O / gate-up / down / LM-head projection, 6 tree attention, 7 RMSNorm,
 * 8 rotary + K/V write, 9 SwiGLU (8 and 9 only where they are kernels of their own: fp32 models),
 * 10 greedy choice and approval, 11 the commit that ends a pass.  The difference between two
 * consecutive marks is the time the earlier kernel added to the pass.  The device keeps the last 16384
 * marks.  end() stops recording, synchronises `stream` and writes the last min(max_marks, kept)
 * marks, oldest first, to out_ns_host / out_kind_host and their number to out_n_host. */
aded_status aded_trace_begin(aded_model* m, void* stream);
aded_status aded_trace_end(aded_model* m, uint64_t* out_ns_host, int32_t* out_kind_host, int32_t max_marks,
                           int32_t* out_n_host, void* stream);

/* Ask the next verify call to also store the residual stream before the first layer and after
 * every layer: hidden_dev receives [n_layers + 1][rows][d_model] in the model dtype.  Lets a checker
 * re-run any single layer from the inputs the device actually had.  Parity checks only. */
aded_status aded_debug_capture_hidden(aded_model* m, void* hidden_dev);

/* Failure-path check ("every device-side wait is bounded", see Conventions): runs one of the library's two
 * kinds of device-side wait -- which = 0: the mbarrier wait of the tensor-core kernels, 1: the wait at an
 * arrival counter of the LM head's tail -- on something that never happens, with a limit of limit_cycles
 * SM clock cycles (1 .. 2^32; about 2 x 10^6 per millisecond).  The wait runs out, the kernel returns, and
 * the model's status word becomes ADED_ERR_TIMEOUT exactly as after a real time-out: later calls do nothing
 * until aded_model_poll_status has read and cleared it.  Nothing faults or hangs.  Asynchronous. */
aded_status aded_debug_wait_timeout(aded_model* m, int32_t which, uint64_t limit_cycles, void* stream);

/* head_dim-128 bf16 models have two tree-attention kernels that compute the same thing with the same
 * rounding points: tcgen05 (which = 0, the default) and mma.sync (which = 1; the kernel head_dim 64
 * always uses).  Selects the one later calls on this model use, so that a test can compare them.
 * ADED_ERR_UNSUPPORTED for models without a tensor-core attention kernel (fp32). */
aded_status aded_debug_attention_kernel(aded_model* m, int32_t which);

/* bf16 models on the tensor-core path keep a private copy of every projection, FFN and LM-head matrix, re-tiled so
 * that each block of the GEMM kernel reads one contiguous run of memory (as many bytes again as those matrices;
 * made once in aded_model_create; when the device has no room for it, the GEMMs read the caller's row-major
 * matrices instead, which is slower).  which = 0: use the copies (the default when they exist;
 * ADED_ERR_UNSUPPORTED when they do not), 1: read the caller's matrices.  Results are identical bit for bit; the
 * switch exists so that a test can say so.  ADED_ERR_UNSUPPORTED for models without the tensor-core GEMM. */
aded_status aded_debug_weight_layout(aded_model* m, int32_t which);

/* Copy out one of the model's activation buffers as the last verify/append call left it (after
 * its last layer): which = 0 residual stream h [rows, d], 1 normalised input x [rows, d], 2 rotated
 * queries q [rows, d], 3 attention output [rows, d], 4 SwiGLU product [rows, F]; model dtype.
 * Stage-by-stage parity checks only. */
aded_status aded_debug_read_buffer(aded_model* m, int32_t which, int32_t rows, void* out_dev, void* stream);

/* Greedy token choice without any allocation.  (The paper has no counterpart of this call; it is
 * the library's per-node greedy choice -- largest fp32 logit, lowest token id among equals -- offered
 * on its own.)
 *
 * For callers that cannot allocate device memory: a process whose device heap is wholly reserved by
 * another component (for instance a framework's caching allocator, so that a cudaMalloc made by this
 * library could fail or stall), or a latency-critical loop that bans allocation calls because
 * cudaMalloc and cudaFree synchronise the device.  Such callers cannot create a model handle, but
 * can still pick tokens from logits they computed elsewhere.
 *   logits_dev    [rows][vocab] fp32, row-major, device memory
 *   out_best_dev  [rows] int32, device memory: index of each row's largest logit
 * The call uses no handle and calls no cudaMalloc, cudaFree or other allocating routine.  Its
 * intermediate results live in a fixed 16 KiB array inside the library's device image (every
 * device that loads the library holds it until the process exits), which bounds the size:
 * rows <= ADED_NOALLOC_MAX_ROWS, otherwise ADED_ERR_INVALID_ARG and nothing is launched.
 * The first call on each device looks up the array's device address (with that device current)
 * and keeps it for the life of the process; make that first call outside any stream capture.  The
 * kept address does not survive cudaDeviceReset or the teardown of the device's primary context --
 * do not call this entry point again in a process that has done either -- and only device ordinals
 * 0..63 are served (ADED_ERR_UNSUPPORTED beyond).  All calls share the one array: it keeps the
 * previous call's contents, which is harmless because every entry is rewritten before it is read,
 * but two calls whose kernels overlap on the GPU (different streams, no dependency) race on it --
 * keep calls on one stream or order them with events.  Work is enqueued on `stream`; the call does
 * not synchronise. */
#define ADED_NOALLOC_MAX_ROWS 128
aded_status aded_greedy_noalloc(const float* logits_dev, int32_t rows, int32_t vocab, int32_t* out_best_dev,
                                void* stream);

/* Read and clear the model's device status word; synchronises `stream`. */
aded_status aded_model_poll_status(aded_model* m, aded_status* out_host, void* stream);

/* ---- tri-gram store (Eq. 1, Algorithm 2) ---------------------------------------------- */

aded_status aded_trigram_create(const aded_trigram_config* cfg, aded_trigram** out);
aded_status aded_trigram_destroy(aded_trigram* t);

/* Algorithm 2 over a token span: every window (tok[i-2], tok[i-1], tok[i]), i = 2 .. n-1, has
 * its count raised by one (saturating at cap), absent tri-grams are inserted with count 1.
 * n < 3 does nothing.  The caller chooses the span; to count a stream piecewise pass each piece
 * with the two tokens that precede it.  A token outside [0, vocab) sets ADED_ERR_INVALID_ARG in
 * the status word and its windows are skipped. */
aded_status aded_trigram_update(aded_trigram* t, const int32_t* tokens_dev, int32_t n, void* stream);
aded_status aded_trigram_update_host(aded_trigram* t, const int32_t* tokens_host, int32_t n, void* stream);

/* For each of q contexts (ctx[2*i], ctx[2*i+1]) the k (1..32) continuations with the largest
 * counts -- equivalently the largest Eq. 1 probabilities -- count descending, token id ascending
 * among equals, padded with token -1 / count 0.  out_total (may be NULL) receives the sum of the
 * context's counts, the denominator of Eq. 1. */
aded_status aded_trigram_topk(const aded_trigram* t, const int32_t* ctx_dev, int32_t q, int32_t k,
                              int32_t* out_tokens_dev, uint32_t* out_counts_dev, uint32_t* out_total_dev,
                              void* stream);
aded_status aded_trigram_topk_host(const aded_trigram* t, const int32_t* ctx_host, int32_t q, int32_t k,
                                   int32_t* out_tokens_host, uint32_t* out_counts_host,
                                   uint32_t* out_total_host, void* stream);

/* Count of one tri-gram (0 if absent); synchronises `stream`.  For tests. */
aded_status aded_trigram_get(const aded_trigram* t, int32_t a, int32_t b, int32_t c,
                             uint32_t* out_count_host, void* stream);
/* Number of stored tri-grams and of buckets in use; synchronises `stream`. */
aded_status aded_trigram_stats(const aded_trigram* t, uint64_t* out_entries_host, uint64_t* out_buckets_host,
                               void* stream);
/* Read and clear the store's device status word; synchronises `stream`. */
aded_status aded_trigram_poll_status(aded_trigram* t, aded_status* out_host, void* stream);

/* ---- keeping and trimming the table (the tri-gram matrix is "initialised from a corpus" and kept
 * between runs; "threshold for the elimination of tri-gram probability", Detailed Experimental
 * Settings) ------------------------------------------------------------------------------------ */

/* Every stored tri-gram whose count is >= min_count: keys_dev[3*i .. 3*i+2] = (w_{i-2}, w_{i-1}, w_i),
 * counts_dev[i] = its count, in no particular order.  *n_out_host = how many there are; only the
 * first max_entries are written (call with max_entries = 0 to size the arrays).  Synchronises. */
aded_status aded_trigram_export(const aded_trigram* t, uint32_t min_count, int32_t* keys_dev, uint32_t* counts_dev,
                                uint64_t max_entries, uint64_t* n_out_host, void* stream);
/* Adds n exported entries to the table: counts of tri-grams already present add up (saturating at
 * the cap).  Asynchronous. */
aded_status aded_trigram_import(aded_trigram* t, const int32_t* keys_dev, const uint32_t* counts_dev, uint64_t n,
                                void* stream);
/* Empties the table (the status word is kept).  Asynchronous. */
aded_status aded_trigram_clear(aded_trigram* t, void* stream);
/* Removes every tri-gram whose count is below min_count and gives its buckets back: the table is
 * rebuilt from the entries that stay.  Allocates a scratch copy of them; synchronises. */
aded_status aded_trigram_prune(aded_trigram* t, uint32_t min_count, void* stream);
/* Writes / reads the table's entries to / from a file on the host ("ADEDTG01", vocab, entry count,
 * keys, counts; native byte order).  Loading ADDS the file's entries to the table (clear it first for
 * a copy) and refuses a file written for another vocabulary size.  Both synchronise. */
aded_status aded_trigram_save(const aded_trigram* t, const char* path, void* stream);
aded_status aded_trigram_load(aded_trigram* t, const char* path, void* stream);

/* ---- draft retrieval and the decoding step on the device ------------------------------------
 * Figure 1's loop -- update the tri-gram matrix, retrieve candidate continuations from it with the
 * last two tokens of the text, hand them to the model as one prefix-sharing pseudo-sequence
 * ("Draft Construction and Verification"), feed the model's output back -- without a host round
 * trip between its stages. */
#define ADED_DRAFT_MAX_K 8

/* Draft tree of exactly n_nodes (1..ADED_MAX_NODES) nodes for the context
 * (context_dev[0], context_dev[1]) = (second-last, last) token of the text.  Node 0 holds the last
 * token.  Nodes are visited in index order; a visited node of depth < max_depth whose parent holds
 * u and which holds w gets one child per entry of the top-k (k in 1..ADED_DRAFT_MAX_K) list of
 * context (u, w), in rank order, appended at the end, until the tree is full: indices are
 * breadth-first, parents[i] < i, siblings differ.  When the table runs dry the tree is completed
 * from filler_dev[0 .. n_filler) (tokens in [0, vocab), supplied by the caller; the paper has no
 * such step, it keeps the launch shape constant): nodes are visited round-robin and a visited
 * node with depth < max_depth and fewer than k children gets the next filler token none of its
 * children holds (tokens passed over are consumed).
 * Outputs (device): tree_tokens[n_nodes], tree_parents[n_nodes], n_from_table[1] (may be NULL):
 * how many nodes came from the table.  If the filler runs out or no node has room left the
 * store's status word becomes ADED_ERR_INVALID_ARG and tree_tokens[0] is set to -1, which the
 * verification step rejects.  Asynchronous on `stream`. */
aded_status aded_draft_tree(const aded_trigram* t, const int32_t* context_dev, int32_t n_nodes, int32_t max_depth,
                            int32_t k, const int32_t* filler_dev, int32_t n_filler, int32_t* tree_tokens_dev,
                            int32_t* tree_parents_dev, int32_t* n_from_table_dev, void* stream);

/* The draft maker of the paper: Monte Carlo tree search over tri-gram continuations (Eq. 2-3,
 * Algorithm 1) from the context (context_dev[0], context_dev[1]).  `iterations` (1..160; the paper
 * uses 150) rounds of selection by the PUCT score with constants c1, c2 (32 and 8 in the paper),
 * expansion of all candidate words of the reached node (its top-k list, k in 1..ADED_DRAFT_MAX_K),
 * simulation up to `length` (1..8; the paper: 4) tokens after the root by drawing from top-k lists in
 * proportion to the counts with the uniform numbers u_dev[iteration * length + draw] (float32 in
 * [0, 1), supplied by the caller), and back propagation of 1 + the sum of the state's Eq. 1
 * probabilities.  The leaves of the search tree are ranked by mean score (earlier-created first on
 * ties); the best n_candidates (the paper: 24; n_candidates * length + 1 <= ADED_MAX_NODES) are
 * written as sentence_tokens_dev[r][length] (-1 padded) with sentence_scores_dev[r], and merged
 * into one prefix tree tree_tokens_dev / tree_parents_dev (breadth-first, *n_nodes_dev nodes, node 0
 * the last token of the text) ready for aded_verify.  With n_nodes_target > 0 the prefix tree is then
 * completed to exactly that many nodes from filler_dev[0 .. n_filler) by the rule of aded_draft_tree
 * (depth limit `length`, at most k children), so that verification steps keep one shape; a filler
 * that runs out is reported as there.  All scores are IEEE doubles computed one rounded operation
 * at a time.  One warp; asynchronous on `stream`. */
aded_status aded_mcts_draft(const aded_trigram* t, const int32_t* context_dev, int32_t iterations, int32_t length,
                            int32_t n_candidates, int32_t k, float c1, float c2, const float* u_dev, int32_t* tree_tokens_dev,
                            int32_t* tree_parents_dev, int32_t* n_nodes_dev, int32_t* sentence_tokens_dev,
                            double* sentence_scores_dev, int32_t* n_sentences_dev, int32_t n_nodes_target,
                            const int32_t* filler_dev, int32_t n_filler, void* stream);

/* aded_decode_step with the draft tree made by aded_mcts_draft (the paper's own loop: tree search over
 * the tri-gram statistics, tree verification, feedback of the output into the statistics), completed
 * to n_nodes nodes with the filler.  u_dev holds iterations * length uniform numbers for this step. */
aded_status aded_decode_step_mcts(aded_model* m, aded_kv* kv, aded_trigram* t, int32_t* context_dev, int32_t n_nodes,
                                  int32_t iterations, int32_t length, int32_t n_candidates, int32_t k, float c1, float c2,
                                  const float* u_dev, const int32_t* filler_dev, int32_t n_filler, int32_t* out_tokens_dev,
                                  int32_t* out_accept_len_dev, void* stream);

/* One decoding step, all on the device and asynchronous on `stream`:
 *   aded_draft_tree from context_dev  ->  aded_verify (out_tokens_dev[n_nodes], out_accept_len_dev[1])
 *   ->  aded_trigram_update over (context, emitted tokens)  ->  context_dev <- last two tokens of the
 *   text after the step.
 * A step whose verification failed (status word of the model set) emits nothing, leaves the cache,
 * the table and the context as they were and writes accept length 0.  n_nodes <= max_rows.
 * n_from_table_dev may be NULL. */
aded_status aded_decode_step(aded_model* m, aded_kv* kv, aded_trigram* t, int32_t* context_dev, int32_t n_nodes,
                             int32_t max_depth, int32_t k, const int32_t* filler_dev, int32_t n_filler,
                             int32_t* out_tokens_dev, int32_t* out_accept_len_dev, int32_t* n_from_table_dev,
                             void* stream);
/* Same with the filler, the emitted tokens and the accept length in host memory (pinned for the
 * copies to be asynchronous); n_filler <= 4 * ADED_MAX_NODES; returns after `stream` has finished. */
aded_status aded_decode_step_host(aded_model* m, aded_kv* kv, aded_trigram* t, int32_t* context_dev, int32_t n_nodes,
                                  int32_t max_depth, int32_t k, const int32_t* filler_host, int32_t n_filler,
                                  int32_t* out_tokens_host, int32_t* out_accept_len_host, void* stream);

const char* aded_status_string(aded_status s);

#ifdef __cplusplus
}
#endif
#endif /* ADED_H */
