/*
 * afx.h -- C ABI of libafx: active-weight selection and sparse GEMV for batch-1 /
 * few-token LLM decoding on NVIDIA B200 (sm_100a), after ActiveFlow (arXiv 2504.08378).
 *
 * Conventions shared by every entry point
 *   - Plain C.  Every pointer says whether it is a HOST or a DEVICE pointer.  The caller
 *     owns every buffer; the library allocates nothing on the calls below unless the
 *     function's comment says so (descriptor create/destroy only).
 *   - `stream` is a cudaStream_t passed as void* (NULL = the default stream).  Calls only
 *     enqueue work on that stream and return; they never synchronise.  Arguments are
 *     validated on the host before anything is launched: on a non-zero return nothing
 *     was enqueued.
 *   - 16-bit floats are passed as raw bit patterns.  dtype AFX_F16 = IEEE binary16,
 *     AFX_BF16 = bfloat16.  Accumulation is always fp32.
 *   - An operator W in R^{N x K} (K input channels, N outputs) is stored
 *     channel-contiguous: channel j is the run Wt[j*ldw .. j*ldw + N).  Wt must be 16-byte
 *     aligned, N % 8 == 0 and ldw % 8 == 0 (so every channel starts on a 16-byte boundary
 *     and can be read with 128-bit loads), ldw >= N.
 *   - An active list is `idx[0..*count)`, int32 channel ids in strictly ascending order,
 *     with the count in DEVICE memory so that no host round trip sits between selection
 *     and the GEMV.
 *   - `dev_status` (where an entry point has it) is a DEVICE int32 or NULL.  Lists and counts
 *     that a kernel reads from caller memory cannot be validated on the host, so the kernels
 *     check them: a count outside [0, K] is clamped (AFX_ERR_CAPACITY), a channel id outside
 *     [0, K) is skipped (AFX_ERR_INVALID_ARG), a negative cache slot is skipped
 *     (AFX_ERR_CAPACITY: the cache ran out of staging rows).  Nothing traps and no address
 *     outside the caller's buffers is formed; the first such event stores its code into
 *     *dev_status if that still holds 0.  The library never clears the word.
 *   - Nothing in the paper prescribes this interface; where an entry point or a parameter is
 *     this library's own device rather than the paper's, its comment says so.
 */
#ifndef AFX_H
#define AFX_H

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef int32_t afx_status;

#define AFX_OK 0
#define AFX_ERR_INVALID_ARG 1 /* NULL required pointer, size out of range */
#define AFX_ERR_ALIGNMENT 2   /* base pointer / N / ldw break the 16-byte rules above */
#define AFX_ERR_CAPACITY 3    /* a caller-provided buffer or a fixed limit is too small */
#define AFX_ERR_UNSUPPORTED 4 /* unknown dtype or mode */
#define AFX_ERR_CUDA 5        /* the CUDA runtime refused a launch or a query */
#define AFX_ERR_TIMEOUT 6     /* reserved: a bounded device-side wait gave up.  No kernel of this */
                              /* version waits on a flag, so nothing returns or stores it.        */

#define AFX_F16 0
#define AFX_BF16 1

#define AFX_MODE_TOPK 0      /* keep the k channels of largest |x|, ties to the lower index */
#define AFX_MODE_THRESHOLD 1 /* keep channels with |x| > tau (strict); tau < 0 keeps all   */

#define AFX_MAX_T 8 /* most tokens per call (few-token decode) */

/* Library version.  HOST pointers; either may be NULL. */
afx_status afx_version(int* major, int* minor);

/* Static, human-readable name of a status code (HOST string, never NULL). */
const char* afx_status_string(afx_status s);

/*
 * Bytes of DEVICE scratch memory the entry points below need for operators of up to K_max
 * channels, N_max outputs and T_max tokens: always 0.  Partial sums meet in shared memory and
 * in the distributed shared memory of a thread-block cluster, and the selection runs inside
 * the consuming kernel, so no call takes a workspace pointer.  (Interface bookkeeping; the
 * paper has no counterpart.)
 */
size_t afx_workspace_bytes(int K_max, int N_max, int T_max);

/*
 * Active-channel selection ("Top-K" operation T of the swapping pipeline, Sec. 4; the
 * magnitude rule of Sec. 2.1; the index-generating kernel of Sec. 6 "Caching").
 *
 *   x        DEVICE, [T][K] 16-bit floats, token-major, 2-byte aligned.
 *   mode     AFX_MODE_TOPK: per token the k largest |x_j| (0 <= k <= K); equal magnitudes
 *            are ranked by ascending channel id.  Magnitudes are compared as the 15-bit
 *            integer "bit pattern with the sign cleared" (NaN patterns therefore rank above
 *            infinity).  AFX_MODE_THRESHOLD: per token the channels with (float)|x_j| > tau;
 *            NaN never passes; tau < 0 keeps every channel.
 *   T > 1    the result is the union of the per-token sets.
 *   idx      DEVICE, capacity K int32; receives the active ids ascending.
 *   count    DEVICE, one int32; receives the number of active ids.
 *   bitmap   DEVICE or NULL; if given, ceil(K/32) uint32 words receive the set as a bitmap
 *            (bit j%32 of word j/32), the form afx_diff_active consumes.
 * 1 <= T <= AFX_MAX_T, 1 <= K <= 2^20.
 */
afx_status afx_select_active(const void* x, int dtype, int K, int T, int mode, int k, float tau,
                             int32_t* idx, int32_t* count, uint32_t* bitmap, void* stream);

/*
 * Cross-layer bookkeeping (Sec. 3: an earlier layer's activation predicts this layer's
 * active set; what the prediction missed is fetched on demand).  A = idxA[0..*cntA) is the
 * actual set, P the predicted set given as a bitmap.  Writes miss = A \ P ascending
 * (capacity K), *miss_count = |A \ P| and *hit_count = |A & P|.  All pointers DEVICE, 4-byte
 * aligned.  An entry of A outside [0, K) counts as neither (see dev_status above).
 */
afx_status afx_diff_active(const int32_t* idxA, const int32_t* cntA, const uint32_t* bitmapP,
                           int K, int32_t* miss, int32_t* miss_count, int32_t* hit_count,
                           int32_t* dev_status, void* stream);

/*
 * Sparse GEMV over the active channels (operation C of the pipeline; Sec. 2.1: only the
 * active elements of the activation take part in the operator):
 *
 *     y[t][i] (+)= sum_{c < *count} x[t][idx[c]] * Wt[col(c)*ldw + i],   0 <= i < N, t < T
 *
 * with col(c) = idx[c], or slot[c] when `slot` is given (the columns then live in a cache
 * whose slot list afx_cache_fetch produced).  Products are exact in fp32; sums are fp32 in
 * a fixed order (same inputs on the same device give the same bits).  One token is multiplied
 * on the fp32 pipe; with 2..8 tokens the active rows are gathered into shared memory and
 * multiplied on the tensor cores (16-bit inputs, fp32 accumulation): the order of the sums, and
 * with it the last bits of y, differ between the two, the rules above hold for both.
 *
 *   Wt        DEVICE, channel-contiguous weights (see the conventions above).
 *   x         DEVICE, [T][K] 16-bit floats; every token uses the whole list.
 *   idx,count DEVICE; an entry outside [0,K) contributes nothing (see dev_status above).
 *   slot      DEVICE int32[*count] or NULL; a negative slot contributes nothing (afx_cache_fetch
 *             writes -1 for a channel it could not place), an upper bound is the caller's to keep
 *             (the kernel does not know how many rows Wt has when it is a cache).
 *   y         DEVICE, [T][N] fp32, 16-byte aligned.  accumulate = 0 overwrites, 1 adds.
 *   dev_status DEVICE int32 or NULL.
 * Needs no scratch memory.  N <= 4 194 240.
 */
afx_status afx_sparse_gemv(const void* Wt, int dtype, int K, int N, int64_t ldw, const void* x,
                           int T, const int32_t* idx, const int32_t* count, const int32_t* slot,
                           float* y, int accumulate, int32_t* dev_status, void* stream);

/*
 * Selection and sparse GEMV in ONE kernel (the T and C operations of Sec. 4 back to back):
 * the result equals afx_select_active followed by afx_sparse_gemv on the same arguments,
 * without the list's round trip through global memory between two launches.  The paper runs T
 * and C as separate pipeline stages; fusing them, and the `kth_hint` slot, are this library's
 * own design for a GPU (the hint is an accelerator only: the paper's thresholds are calibrated
 * offline, here the exact top-k search merely starts near the previous answer).
 *
 *   Wt, x, y, accumulate   as for afx_sparse_gemv;  mode, k, tau  as for afx_select_active.
 *   idx_out   DEVICE int32[K] or NULL: receives the active list.
 *   count_out DEVICE int32[1] or NULL: receives its length.
 *   kth_hint  DEVICE int32[1] or NULL, read and rewritten by a top-k call with T == 1 and
 *             0 < k < K: on return 0x10000 | the k-th largest magnitude key (the 16-bit pattern
 *             with the sign cleared).  A value with bit 16 set that a call finds there is where
 *             its search for the k-th key starts (cheap when the key lies within about 19 % of
 *             it, e.g. the previous token's key for the same operator; the full search
 *             otherwise); 0 means no hint.  The selected set never depends on it.
 * K * T * 2 bytes of x are read by every thread block (they stay in L2).
 */
afx_status afx_select_gemv(const void* Wt, int dtype, int K, int N, int64_t ldw, const void* x, int T,
                           int mode, int k, float tau, float* y, int accumulate, int32_t* idx_out,
                           int32_t* count_out, int32_t* kth_hint, void* stream);

/*
 * The same sparse GEMV over 4-bit block-quantised weights (the storage type of every model the
 * paper evaluates, Sec. 7.1; Sec. 6: the weights are transposed so that a channel's scaling
 * factors are read together with the channel).  Channel j is the row Wq[j * ldq_bytes ..):
 * N/2 bytes of 4-bit codes, then N/32 fp16 scales; a block of 32 outputs b has 16 code bytes --
 * byte m holds the code of output 32b + m in its low 4 bits and of output 32b + 16 + m in its
 * high 4 bits -- and one scale; value = (code - 8) * scale (the block format of llama.cpp's
 * 4-bit type with the scales moved behind the codes, so that both parts keep 16-byte alignment).
 *
 *   Wq         DEVICE, 16-byte aligned; N % 32 == 0; ldq_bytes % 16 == 0, >= afx_q4_row_bytes(N).
 *   x          DEVICE [K] 16-bit floats of type x_dtype (one token).
 *   idx,count,dev_status   as for afx_sparse_gemv;  y DEVICE [N] fp32.
 * fp32 accumulation in a fixed order.
 */
size_t afx_q4_row_bytes(int N); /* bytes of one channel row without padding beyond 16 (0: bad N) */
afx_status afx_sparse_gemv_q4(const void* Wq, int K, int N, int64_t ldq_bytes, const void* x, int x_dtype,
                              const int32_t* idx, const int32_t* count, float* y, int accumulate,
                              int32_t* dev_status, void* stream);

/* ------------------------------------------------------------------------------------------
 * Decoder layers: every linear operator of a Llama-shaped layer run as ONE kernel that
 * normalises (where the layer does), selects the active channels of its own input and
 * evaluates the operator on them -- the paper's per-operator T (Top-K) + C (compute) pair of
 * Sec. 4 applied "to all linear transformation operators" (Sec. 2.1), with the cross-layer
 * prediction and miss bookkeeping of Sec. 3.  Attention itself stays dense.
 * ------------------------------------------------------------------------------------------ */

typedef struct afx_model afx_model; /* opaque, HOST object */
typedef struct afx_state afx_state; /* opaque, HOST object describing a DEVICE blob */

/* The four distinct operator inputs of a layer (q, k and v share one; gate and up share one). */
#define AFX_OP_QKV 0  /* input: RMSNorm(h) * g_attn        -> q | k | v          */
#define AFX_OP_O 1    /* input: attention output           -> h += W_o a         */
#define AFX_OP_GU 2   /* input: RMSNorm(h) * g_mlp         -> silu(gate) * up    */
#define AFX_OP_DOWN 3 /* input: silu(gate) * up            -> h += W_down hm     */

#define AFX_XL_OFF 0      /* no cross-layer prediction                                         */
#define AFX_XL_BOOKKEEP 1 /* paper: compute on the actual set A; the set P predicted by an    */
                          /* earlier layer only decides what was preloaded; A \ P is listed    */
#define AFX_XL_REUSE 2    /* compute on the predicted set P, no selection in predicted layers  */

typedef struct {
    int32_t dtype;       /* AFX_F16 / AFX_BF16: weights and rounded activations               */
    int32_t n_layers;
    int32_t hidden;      /* model width; multiple of 8                                         */
    int32_t n_heads;     /* query heads                                                        */
    int32_t n_kv_heads;  /* divides n_heads, n_heads / n_kv_heads <= 8                         */
    int32_t head_dim;    /* must be 128                                                        */
    int32_t mlp;         /* MLP width; multiple of 8                                           */
    int32_t max_seq;     /* rows of each KV cache; positions 0 .. max_seq-1                    */
    float rms_eps;
    float rope_theta;
    int32_t select_mode; /* AFX_MODE_TOPK / AFX_MODE_THRESHOLD                                 */
    int32_t xl_depth;    /* d: layers p = 0, d, 2d, .. predict layers p+1 .. p+d; 0 = off      */
    int32_t xl_mode;     /* AFX_XL_*                                                           */
} afx_model_desc;

typedef struct {
    /* DEVICE pointers, channel-contiguous (see the conventions at the top), 16-byte aligned.  */
    /* A weight pointer may be NULL when that operator is always given another way (host       */
    /* handles, 4-bit rows); a step that needs it then returns AFX_ERR_INVALID_ARG.            */
    const void* w_qkv;  /* [hidden][(n_heads + 2 n_kv_heads) * 128]  columns: q | k | v        */
    const void* w_o;    /* [n_heads * 128][hidden]                                             */
    const void* w_gu;   /* [hidden][2 * mlp]: columns in groups of 16 = gate[8m..8m+8) then    */
                        /* up[8m..8m+8), so that one pass yields silu(gate) * up               */
    const void* w_down; /* [mlp][hidden]                                                       */
    const float* g_attn; /* [hidden] fp32 RMSNorm gains                                        */
    const float* g_mlp;
    void* k_cache;      /* [T][max_seq][n_kv_heads][128] fp16, one cache per token stream      */
    void* v_cache;
    int32_t k[4];       /* per AFX_OP_*: channels kept in top-k mode                           */
    float tau[4];       /* per AFX_OP_*: threshold in threshold mode                           */
} afx_layer_desc;

/*
 * Creates the HOST-side model object: copies both descriptor arrays (layers[n_layers]) and
 * allocates one small DEVICE table (rotary cos/sin, 512 * max_seq bytes) with cudaMalloc.
 * Weights and caches stay the caller's.  afx_model_destroy frees the table and the object.
 */
afx_status afx_model_create(const afx_model_desc* desc, const afx_layer_desc* layers, afx_model** out);
afx_status afx_model_destroy(afx_model* model);

/*
 * (The state object and its accessors are this library's own plumbing; the paper has no
 * counterpart.)
 * Per-sequence working set for T token streams decoded together (1 <= T <= AFX_MAX_T): the
 * fp32 residual h[T][hidden], the operators' intermediate vectors, the current and predicted
 * active sets of the four operator inputs, and per-layer counters.  The caller allocates
 * afx_state_bytes() of DEVICE memory (256-byte aligned); afx_state_create clears it on
 * `stream` and returns a HOST handle that only records where things live in the blob.
 */
size_t afx_state_bytes(const afx_model* model, int T);
afx_status afx_state_create(const afx_model* model, int T, void* blob, size_t bytes, void* stream,
                            afx_state** out);
afx_status afx_state_destroy(afx_state* state);

/* Buffers inside the state blob (DEVICE addresses), for loading h and reading results back. */
#define AFX_BUF_H 0          /* fp32 [T][hidden]      residual stream, input and output       */
#define AFX_BUF_QKV 1        /* fp32 [T][n_qkv]       q | k | v before rotation               */
#define AFX_BUF_ATTN 2       /* dtype [T][n_heads*128] attention output (input of W_o)         */
#define AFX_BUF_HM 3         /* dtype [T][mlp]        silu(gate)*up (input of W_down)          */
#define AFX_BUF_XNORM 4      /* dtype [T][hidden]     op = AFX_OP_QKV or AFX_OP_GU: normed input */
#define AFX_BUF_IDX 5        /* int32 [K_op]          active list last used by operator input `op` */
#define AFX_BUF_MISS 6       /* int32 [K_op]          A \ P of the last bookkeeping            */
#define AFX_BUF_STATS 7      /* int32 [n_layers][4][4] per layer and op: list length, |A & P|,  */
                             /*                       |A \ P| (written by each layer step), and */
                             /*                       0x10000 | the k-th largest magnitude key  */
                             /*                       of the last one-token top-k selection (0  */
                             /*                       before the first; the next token's search */
                             /*                       starts there, any value gives the same set) */
#define AFX_BUF_HINTS 8      /* int32 [n_layers][4][AFX_MAX_T] the same search hints per token when T > 1: */
                             /*                       0x10000 | k-th key of token t's last selection   */
afx_status afx_state_buffer(const afx_state* state, int which, int op, void** ptr, size_t* bytes);

/*
 * One decoder layer for the T token streams at position `pos` (0 <= pos < max_seq; the
 * cache rows 0..pos-1 hold the past, row pos is written): five kernels on `stream`,
 *   qkv (RMSNorm + select + GEMV) -> rotary, cache append, dense attention ->
 *   o (select + GEMV, h +=) -> gate/up (RMSNorm + select + GEMV + silu*up) ->
 *   down (select + GEMV, h +=).
 * Layers must be stepped in order 0 .. n_layers-1 when cross-layer prediction is on.
 */
afx_status afx_layer_step(afx_model* model, int layer, afx_state* state, int pos, void* stream);

/*
 * ONE of the five kernels of afx_layer_step, on whatever the state holds (afx_layer_step is
 * exactly the five calls in order).  For per-operator timing and profiling of the launches a
 * decode step really makes -- the same kernel instantiation, launch shape and side outputs;
 * this library's own addition, the paper has no counterpart.
 */
#define AFX_STEP_QKV 0
#define AFX_STEP_ATTN 1
#define AFX_STEP_O 2
#define AFX_STEP_GU 3
#define AFX_STEP_DOWN 4
afx_status afx_layer_kernel(afx_model* model, int layer, afx_state* state, int pos, int which, void* stream);

/*
 * The MLP block alone on a given (already normalised) input: y = W_down(silu(W_gate x) * W_up x)
 * with both selections; x DEVICE [T][hidden] dtype, y DEVICE [T][hidden] fp32 (overwritten).
 * Uses the state's HM buffer and active-set buffers; no cross-layer prediction.
 */
afx_status afx_mlp_block(afx_model* model, int layer, afx_state* state, const void* x, float* y,
                         void* stream);

/* ------------------------------------------------------------------------------------------
 * Hot-weight cache (Sec. 4.2 "Dynamic LLM Weight Caching": per weight tensor a table from
 * channel to cache slot and a usage count per channel that starts from zero with every new
 * sequence; a newly active channel replaces the least used cached one).  The full operator
 * lives in pinned HOST memory (standing in for flash); the cache holds `capacity` of its
 * channels in DEVICE memory.  afx_cache_fetch takes one step's active list, counts the usage,
 * decides hits / replacements, copies every missed channel from the host into its slot and
 * returns the slot of each active channel, which afx_sparse_gemv accepts as its `slot` list.
 *
 * Policy, for the ascending active list of one step:
 *   1. count[j] += 1 for every active j;  2. a channel that already has a slot is a hit;
 *   3. misses in ascending channel order: the lowest free slot if there is one; otherwise the
 *      cached channel that is NOT active in this step with the smallest (count, channel id) is
 *      the victim and is replaced when count[miss] >= count[victim] (the paper's worked example
 *      replaces on equal counts); a miss that replaces nothing is "transient": it is copied
 *      into staging row capacity + r (r = its rank among this step's transients), used for
 *      this step and not retained.
 * ------------------------------------------------------------------------------------------ */

typedef struct afx_cache afx_cache; /* opaque, HOST object owning small DEVICE tables */

typedef struct {
    int32_t dtype;         /* AFX_F16 / AFX_BF16                                                 */
    int32_t K, N;          /* channels of the operator, values per channel (N % 8 == 0)          */
    int64_t ldw;           /* row stride in elements of BOTH host_base and slots (ldw % 8 == 0)  */
    int32_t capacity;      /* cached channels C, 1 <= C <= K                                     */
    int32_t staging_rows;  /* rows after the C cache rows for transient channels (>= 0)          */
    const void* host_base; /* HOST, [K][ldw], page-locked (cudaHostAlloc / cudaHostRegister)     */
    void* slots;           /* DEVICE, [C + staging_rows][ldw], 16-byte aligned, caller-owned     */
} afx_cache_desc;

typedef struct {
    int32_t hits, misses, transients; /* of the last afx_cache_fetch                            */
    int32_t overflow;                 /* transients that did not fit into staging_rows (their   */
                                      /* slot is -1: the step's result must not be used)        */
    uint64_t bytes_fetched;           /* host -> device bytes of the last fetch: copied * N * 2 */
} afx_cache_stats;

/*
 * afx_cache_create checks the descriptor, resolves the device view of host_base (returns
 * AFX_ERR_INVALID_ARG when it is not page-locked) and allocates the tables (cudaMalloc:
 * slot per channel, channel per slot, count per channel, work lists; about 24 bytes per
 * channel).  The cache starts empty.  afx_cache_destroy frees them.
 */
afx_status afx_cache_create(const afx_cache_desc* desc, afx_cache** out);
afx_status afx_cache_destroy(afx_cache* cache);

/* New sequence: every usage count returns to zero; cached channels stay.  Enqueued on stream. */
afx_status afx_cache_reset(afx_cache* cache, void* stream);

/* Pre-load channels (HOST list, n <= free slots, not yet cached) into the lowest free slots,
 * copying their columns; used to set the initial cache contents.  Synchronises the stream. */
afx_status afx_cache_install(afx_cache* cache, const int32_t* host_channels, int n, void* stream);

/*
 * One step.  idx / count: DEVICE active list (ascending; as afx_select_active writes it).
 * slot_out: DEVICE int32[K]; entry c receives the row of idx[c] in `slots` (-1 for a transient
 * that found no staging row, and for an entry outside [0, K), which takes no part in the
 * step).  stats: DEVICE afx_cache_stats or NULL.  dev_status: DEVICE int32 or NULL (see the
 * conventions at the top; staging overflow stores AFX_ERR_CAPACITY, and afx_sparse_gemv then
 * leaves the unplaced channels out instead of reading a row that does not exist).  Two
 * kernels on `stream`: the policy (one thread block; the victims are ordered by a bitonic
 * sort of (count, channel) keys) and the copy of the missed channels (128-bit loads from the
 * mapped host memory).  No host synchronisation.
 */
afx_status afx_cache_fetch(afx_cache* cache, const int32_t* idx, const int32_t* count, int32_t* slot_out,
                           afx_cache_stats* stats, int32_t* dev_status, void* stream);

/* Copies the tables to HOST arrays for inspection (either may be NULL): slot_of[K] (-1 = not
 * cached), usage[K].  Synchronises the stream. */
afx_status afx_cache_snapshot(afx_cache* cache, int32_t* host_slot_of, uint32_t* host_usage, void* stream);

/* ------------------------------------------------------------------------------------------
 * Cross-layer-group weight swapping (Sec. 3 "Cross-layer Active Weight Preloading" with its
 * data layout, and the PL "preload" / L "on-demand load" operations of the pipeline of Sec. 4).
 * One object serves ONE operator type (say W_down) of all layers.  Its weights live in pinned
 * HOST memory in the paper's reordered layout: groups of `group` consecutive layers (group g =
 * layers g*group .. g*group+group-1, the last one possibly shorter); inside a group the columns
 * are ordered by channel id, then layer id -- [Ch0_L, Ch0_L+1, .., Ch1_L, Ch1_L+1, ..] -- so
 * the columns one predicted channel needs in all layers of the group are ONE contiguous chunk.
 *
 * While the layers of a group are computed, afx_swap_preload copies the chunks of the channels
 * PREDICTED for the next group (the active list of an earlier layer's activation) into device
 * rows on a loader stream; when a layer's actual activation is known, afx_swap_acquire maps
 * every active channel to its preloaded row or loads it on demand (one column, this layer
 * only) and returns the slot list that afx_sparse_gemv takes.  Stream events stand in for the
 * paper's request / complete signals between the loading and the computing thread; no kernel
 * spins on a flag.
 * ------------------------------------------------------------------------------------------ */

typedef struct afx_swap afx_swap; /* opaque, HOST object owning small DEVICE tables, two pairs of events and
                                     (unless one is given) a loader stream */

typedef struct {
    int32_t dtype;        /* AFX_F16 / AFX_BF16                                                  */
    int32_t n_layers;     /* layers that have this operator                                      */
    int32_t group;        /* d: layers per cross-layer group (>= 1)                              */
    int32_t K, N;         /* channels of the operator, values per channel (N % 8 == 0)           */
    int64_t ldw;          /* row stride in elements of the host image AND the device rows        */
    int32_t rows_pred;    /* device rows per layer for preloaded channels (a longer prediction   */
                          /* is cut: its first rows_pred channels are preloaded)                 */
    int32_t rows_miss;    /* device rows per layer for on-demand channels                        */
    const void* host_base;/* HOST, page-locked, n_layers * K rows of ldw in the group layout     */
    void* dev_rows;       /* DEVICE, afx_swap_device_bytes() bytes, 16-byte aligned:             */
                          /* [2 buffers][group][rows_pred + rows_miss][ldw]; groups alternate    */
    void* loader_stream;  /* cudaStream_t the preloads run on, or NULL: the object creates one   */
} afx_swap_desc;

typedef struct {
    int32_t hits;      /* active channels found preloaded                                        */
    int32_t ondemand;  /* active channels loaded on demand by this acquire                       */
    int32_t overflow;  /* active channels that found no on-demand row (slot -1)                  */
    int32_t preloaded; /* channels the group's preload brought in                                */
    uint64_t bytes_preload;  /* host -> device bytes of that preload (preloaded * layers * N * 2) */
    uint64_t bytes_ondemand; /* host -> device bytes of this acquire (ondemand * N * 2)          */
} afx_swap_stats;

/* Element offset of column (layer, channel) in the host image (HOST arithmetic, no GPU needed);
 * (size_t)-1 for arguments out of range. */
size_t afx_swap_host_offset(int n_layers, int group, int K, int64_t ldw, int layer, int channel);

/* Re-orders per-layer operator tensors (HOST pointers per_layer[l] -> [K][ldw] 16-bit values)
 * into the group layout at host_out (n_layers * K * ldw values).  Plain host copies. */
afx_status afx_swap_pack_host(const void* const* per_layer, int n_layers, int group, int K, int64_t ldw,
                              void* host_out);

/* Bytes of dev_rows the descriptor needs (0 for a bad descriptor). */
size_t afx_swap_device_bytes(const afx_swap_desc* desc);

/* Resolves the device view of host_base (AFX_ERR_INVALID_ARG when it is not page-locked),
 * allocates the tables (cudaMalloc, about 20 bytes per channel), creates the events and, if
 * none was given, the loader stream.  afx_swap_destroy releases them. */
afx_status afx_swap_create(const afx_swap_desc* desc, afx_swap** out);
afx_status afx_swap_destroy(afx_swap* swap);

/*
 * PL: preload group `group_index` from the predicted list idxP[0 .. *cntP) (DEVICE, ascending, as
 * afx_select_active or a layer step writes it).  Enqueued on the loader stream behind everything
 * enqueued on compute_stream so far (the list must have been produced there; idxP must hold K
 * readable entries: the call first takes its own copy on compute_stream, so the caller may
 * overwrite the list afterwards); predicted channel c goes to row c of every layer of the group.  copy_blocks: thread blocks of the copy
 * kernel (0 = 32; it reads host memory over PCIe and needs few).  Call it only after the
 * compute stream has been given all work of group_index - 2, whose buffer it overwrites.
 */
afx_status afx_swap_preload(afx_swap* swap, int group_index, const int32_t* idxP, const int32_t* cntP,
                            int copy_blocks, int32_t* dev_status, void* compute_stream);

/*
 * L: the layer's actual active list idxA[0 .. *cntA) is known.  On compute_stream: waits for the
 * preload of the layer's group (if one was requested; otherwise nothing counts as preloaded),
 * writes slot_out[c] = row of idxA[c] (preloaded row, or rows_pred + m for the m-th on-demand
 * channel, or -1 when the on-demand rows are used up: AFX_ERR_CAPACITY in dev_status, and
 * afx_sparse_gemv leaves such channels out), copies the on-demand columns, fills *stats
 * (DEVICE or NULL).  *rows_out (HOST) receives the DEVICE address of this layer's rows: pass it
 * as Wt, with slot_out as slot, to afx_sparse_gemv on the same stream.
 */
afx_status afx_swap_acquire(afx_swap* swap, int layer, const int32_t* idxA, const int32_t* cntA,
                            int32_t* slot_out, afx_swap_stats* stats, int32_t* dev_status, void* compute_stream,
                            const void** rows_out);

/* ------------------------------------------------------------------------------------------
 * Cost model of the swapping pipeline and the greedy parameter search (Sec. 4.1 "Elastic and
 * Optimized LLM Execution", Eq. 1-9 and the symbol table).  HOST arithmetic; sizes in bytes,
 * bandwidths in bytes per second, times in seconds.
 * ------------------------------------------------------------------------------------------ */

typedef struct {
    double sp;             /* sparsity of the model                                            */
    double hr;             /* average hit rate of the weight cache                             */
    double si;             /* average similarity inside a cross-layer group                    */
    int32_t N;             /* layers per cross-layer group                                     */
    int32_t n_layers;      /* layers of the model (0: T_token counts two groups)               */
    double S_l;            /* size of one layer                                                */
    double bw_mem;         /* BW_mem                                                           */
    double bw_flash_small; /* BW_flash^small: single-channel reads (on-demand loads)           */
    double bw_flash_large; /* BW_flash^large: group-chunk reads (preloads)                     */
    double M_cache, M_kv;  /* memory of the weight cache and of the KV cache                   */
} afx_cost_params;

typedef struct {
    double M_cl;      /* Eq. 9: S_l (1 - sp) N                                                  */
    double M;         /* Eq. 8: M_cl + M_cache + M_kv                                           */
    double T_load;    /* Eq. 3: M_cl (1 - hr) / BW_flash^small                                  */
    double T_comp;    /* Eq. 4: M_cl / BW_mem                                                   */
    double T_onload;  /* Eq. 6: S_l (1 - sp)(1 - hr)(1 - si) / BW_flash^small                   */
    double T_preload; /* Eq. 7: M_cl (1 - hr) / BW_flash^large                                  */
    double T_overlap; /* Eq. 5: T_onload + max(T_preload, T_comp)                               */
    double T_decode;  /* Eq. 1 as printed: T_load + T_overlap + T_comp                          */
    double T_token;   /* the same with one overlap stage per further group of the model:        */
                      /* T_load + (ceil(n_layers / N) - 1) T_overlap + T_comp                   */
} afx_cost;

afx_status afx_cost_eval(const afx_cost_params* params, afx_cost* out);

/* Why the search stopped growing the group. */
#define AFX_COST_STOP_BALANCED 0 /* T_preload <= T_comp: preloading hides behind computation   */
#define AFX_COST_STOP_GAIN 1     /* one more layer lowered T_preload per layer by < min_gain   */
#define AFX_COST_STOP_MEMORY 2   /* a larger group no longer fits M_max                        */
#define AFX_COST_STOP_N_MAX 3    /* N_max (or the layer count) reached                         */

typedef struct {
    double S_m, S_l;             /* size of the model, of one layer                             */
    int32_t n_layers;
    double M_max, M_kv;          /* memory budget; fixed KV-cache memory                        */
    double bw_mem, bw_flash_small;
    int32_t n_chunk;             /* measured large-read bandwidth by chunk size (HOST arrays,   */
    const double* chunk_bytes;   /* chunk_bytes ascending); a group of N layers reads chunks of */
    const double* chunk_bw;      /* N * column_bytes                                            */
    double column_bytes;         /* bytes of one channel of one layer's operator                */
    int32_t n_hr;                /* measured cache hit rate by cache size as a fraction of S_m  */
    const double* hr_cache_frac; /* (HOST arrays, ascending)                                    */
    const double* hr_value;
    double si;                   /* cross-layer similarity                                      */
    double min_gain;             /* relative drop of T_preload per layer that still pays        */
    int32_t N_max;
} afx_cost_search_in;

typedef struct {
    double sp;        /* 1 - M_max / S_m (not below 0)                                          */
    int32_t N;        /* chosen layers per group                                                */
    double M_cache;   /* what the budget leaves for the weight cache                            */
    double hr;        /* hit rate read from the table at that cache size                        */
    double bw_flash_large;
    afx_cost cost;
    int32_t stop_reason;
} afx_cost_choice;

/*
 * The paper's greedy search: sparsity from the memory budget, then the group grows one layer
 * at a time (larger chunks read faster) until preloading is no slower than computing, the
 * gain per added layer falls below min_gain, or the budget is exhausted; the memory a group
 * does not need goes to the weight cache.  AFX_ERR_CAPACITY when even one layer does not fit.
 */
afx_status afx_cost_search(const afx_cost_search_in* in, afx_cost_choice* out);

/* ------------------------------------------------------------------------------------------
 * Mixture-of-experts MLP block for one token (the Mixtral-8x7B deployment of Sec. 1 and the
 * evaluation; the paper applies the same active-weight selection inside every expert).  The
 * router stays dense; each chosen expert's gate|up and down operators run on the active
 * channels of their own input, as in afx_mlp_block:
 *
 *     logits = W_r x;  e_1..e_top = the experts of largest logit (ties: lower id first);
 *     p = softmax(logits[e_1..e_top]);  y (+)= sum_r p_r * W_down[e_r](silu(W_gate[e_r] x) * W_up[e_r] x)
 *
 * The experts are chosen ON THE DEVICE (no host round trip): the kernels take their weights
 * from DEVICE tables of device pointers, indexed by what the router kernel wrote.  Four
 * kernels on `stream`: the router, the chosen experts' gate|up operators side by side in one
 * grid, their down operators likewise (each weighted output in the workspace), and the sum of
 * those outputs in the order of the router's choice.
 * ------------------------------------------------------------------------------------------ */

typedef struct {
    int32_t dtype;        /* AFX_F16 / AFX_BF16                                                  */
    int32_t hidden, mlp;  /* model width, expert MLP width (multiples of 8, <= 32768)            */
    int32_t n_experts;    /* 1 .. 16                                                             */
    int32_t top;          /* experts per token, 1 .. min(4, n_experts)                           */
    int32_t select_mode;  /* AFX_MODE_*: selection inside the experts                            */
    int32_t k_gu, k_down; /* top-k counts of the two expert operators                            */
    float tau_gu, tau_down;
    const void* w_router; /* DEVICE [hidden][ld_router] 16-bit, channel-contiguous, first        */
    int64_t ld_router;    /* n_experts values of a row used (ld_router >= n_experts)             */
    const void* w_gu_table;   /* DEVICE array of n_experts DEVICE pointers: [hidden][2*mlp], the  */
                              /* interleaved gate|up layout of afx_layer_desc, 16-byte aligned   */
    const void* w_down_table; /* DEVICE array of n_experts DEVICE pointers: [mlp][hidden]         */
} afx_moe_desc;

/* Bytes of DEVICE workspace afx_moe_block needs (256-byte aligned): router results, the chosen
 * experts' intermediate vectors and their weighted outputs before they are added up.  0 for a
 * bad descriptor. */
size_t afx_moe_workspace_bytes(const afx_moe_desc* desc);

/*
 *   x   DEVICE [hidden] 16-bit (already normalised);  y DEVICE [hidden] fp32, 16-byte aligned;
 *   accumulate = 0 overwrites y, 1 adds to it (the residual stream).
 * After the call the workspace starts with float logits[16], int32 experts[4], float
 * weights[4] (for inspection).
 */
afx_status afx_moe_block(const afx_moe_desc* desc, const void* x, float* y, int accumulate, void* workspace,
                         size_t workspace_bytes, void* stream);

/*
 * afx_layer_step for a layer some of whose operators do not live in device memory: per
 * operator input (AFX_OP_*) either an LFU cache (afx_cache: THIS layer's operator tensor) or a
 * swapping object (afx_swap: the operator type of all layers).  Such an operator runs as the
 * paper's pipeline stages one after the other on `stream` -- T: input stage + selection (the
 * side outputs of the fused kernel: normed input, active list, cross-layer bookkeeping), L:
 * afx_cache_fetch / afx_swap_acquire, C: the sparse GEMV through the slot list with the
 * operator's epilogue -- while operators with neither handle run fused on the resident weights
 * of the layer descriptor.  slot[op]: DEVICE int32[K_op] scratch for the slot list.  Preloads
 * (afx_swap_preload from the state's AFX_BUF_IDX list) are the caller's to request between layer
 * steps.  AFX_XL_REUSE models are not supported.  q|k|v, gate|up (interleaved) and the
 * other operators use the layouts of afx_layer_desc in their host images.
 */
typedef struct {
    afx_cache* cache[4]; /* per AFX_OP_*: or NULL */
    afx_swap* swap[4];   /* per AFX_OP_*: or NULL (not both)                                      */
    int32_t* slot[4];    /* DEVICE int32[K_op] where a handle is given                            */
} afx_hosted_ops;
afx_status afx_layer_step_hosted(afx_model* model, int layer, afx_state* state, int pos, const afx_hosted_ops* ops,
                                 int32_t* dev_status, void* stream);

/*
 * afx_layer_step for a layer whose operator weights are 4-bit (the storage type of the paper's
 * models, Sec. 7.1; rows as for afx_sparse_gemv_q4): per operator ONE kernel, as in
 * afx_layer_step -- input stage, selection with its side outputs (normed input, active list,
 * cross-layer bookkeeping), the 4-bit sparse GEMV over the selected channels and the operator's
 * epilogue (q|k|v: store; o and down: h +=; gate|up: silu(gate) * up, rounded to the model's
 * 16-bit type).  One token (state T == 1).  An operator whose wq is NULL runs on the 16-bit
 * weights of the layer descriptor.  Cross-layer modes as in afx_layer_step.
 *
 *   wq[op]         DEVICE, 16-byte aligned: K_op rows of ldq_bytes[op] bytes (a multiple of 16,
 *                  >= afx_q4_row_bytes(N_op)); N_op % 32 == 0.  Borrowed for the call.
 *   gate|up        block b of 32 outputs of a row holds gate outputs 16b .. 16b+15 in the low
 *                  4 bits of its 16 bytes and up outputs 16b .. 16b+15 in the high 4 bits: one
 *                  scale serves 16 gate and 16 up weights of the same intermediate channels.
 *   dev_status     reserved (may be NULL; 4-byte aligned): every list this path multiplies by
 *                  comes from its own selection, so no device check can fire.
 */
typedef struct {
    const void* wq[4];    /* per AFX_OP_*: 4-bit rows or NULL */
    int64_t ldq_bytes[4]; /* row stride where wq is given     */
} afx_q4_layer;
afx_status afx_layer_step_q4(afx_model* model, int layer, afx_state* state, int pos, const afx_q4_layer* q4,
                             int32_t* dev_status, void* stream);

/*
 * The MLP block without any allocation (the paper has no counterpart: this entry point exists
 * for the integration, not for the method).  Same result as afx_mlp_block on the same weights
 * and input -- y = W_down(silu(W_gate x) * W_up x), both operators on the active channels of
 * their own input -- but it needs neither afx_model_create (which calls cudaMalloc for its
 * rotary table) nor a caller-allocated state blob: the intermediate vector silu(gate) * up is
 * kept in a fixed array inside the library image (AFX_MAX_T * AFX_NOALLOC_MAX_MLP 16-bit values
 * = 512 KB per GPU, held by every GPU that loads the library until the process exits).  It is
 * meant for callers that must not allocate device memory: a serving process that has handed all
 * of HBM to its own pool, code in a latency-critical loop where cudaMalloc's device-wide
 * synchronisation is not acceptable, or a plug-in that is only given pointers.  The call itself
 * uses no cudaMalloc, cudaFree or other allocating routine.
 *
 *   w_gu    DEVICE [hidden][2*mlp] channel-contiguous, columns in groups of 16 = gate[8m..8m+8)
 *           then up[8m..8m+8) (the w_gu layout of afx_layer_desc); w_down DEVICE [mlp][hidden].
 *   x       DEVICE [T][hidden] 16-bit floats (already normalised); y DEVICE [T][hidden] fp32,
 *           overwritten.  mode, k_*, tau_* as for afx_select_active, per operator.
 * hidden and mlp are multiples of 8; hidden <= 32768; mlp > AFX_NOALLOC_MAX_MLP returns
 * AFX_ERR_CAPACITY and launches nothing.
 * The first call on a device looks up the array's device address (with that device current)
 * and keeps it for the life of the process (it does not survive cudaDeviceReset); make that
 * first call outside any stream capture -- a first call on a capturing stream returns
 * AFX_ERR_INVALID_ARG and launches nothing.  All calls on a device share the array and
 * it keeps the previous call's contents (nothing in it has to start from zero: each call
 * rewrites the T * mlp values it reads): two calls whose kernels overlap on the GPU -- different
 * streams, or graphs replayed concurrently -- race on it; serialise them.
 */
#define AFX_NOALLOC_MAX_MLP 32768
afx_status afx_mlp_block_noalloc(const void* w_gu, const void* w_down, int dtype, int hidden, int mlp,
                                 const void* x, int T, int mode, int k_gu, float tau_gu, int k_down,
                                 float tau_down, float* y, void* stream);

#ifdef __cplusplus
}
#endif
#endif /* AFX_H */
