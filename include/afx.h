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
#define AFX_ERR_TIMEOUT 6     /* a bounded device-side wait gave up (reported via a status word) */

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
 * Scratch memory needed by afx_sparse_gemv for operators of at most N_max outputs and T_max
 * tokens on the current device.  The caller allocates that many bytes of DEVICE memory
 * (256-byte aligned) once, clears it with afx_workspace_init before its first use, and may
 * reuse it for any number of calls that are ordered on one stream.  Two calls that may
 * overlap on the GPU need two workspaces.  Returns 0 on a bad argument.
 */
size_t afx_workspace_bytes(int N_max, int T_max);

/* Enqueue the clearing of a fresh workspace (its split counters must start at zero;
 * every call leaves them at zero again). */
afx_status afx_workspace_init(void* workspace /*DEVICE*/, size_t bytes, void* stream);

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
 * (capacity K), *miss_count = |A \ P| and *hit_count = |A & P|.  All pointers DEVICE.
 */
afx_status afx_diff_active(const int32_t* idxA, const int32_t* cntA, const uint32_t* bitmapP,
                           int K, int32_t* miss, int32_t* miss_count, int32_t* hit_count,
                           void* stream);

/*
 * Sparse GEMV over the active channels (operation C of the pipeline; Sec. 2.1: only the
 * active elements of the activation take part in the operator):
 *
 *     y[t][i] (+)= sum_{c < *count} x[t][idx[c]] * Wt[col(c)*ldw + i],   0 <= i < N, t < T
 *
 * with col(c) = idx[c], or slot[c] when `slot` is given (the columns then live in a cache
 * whose slot list afx_cache_fetch produced).  Products are exact in fp32; sums are fp32 in
 * a fixed order (same inputs give the same bits).
 *
 *   Wt        DEVICE, channel-contiguous weights (see the conventions above).
 *   x         DEVICE, [T][K] 16-bit floats; every token uses the whole list.
 *   idx,count DEVICE; entries must lie in [0,K) (not checked on the device).
 *   slot      DEVICE int32[*count] or NULL.
 *   y         DEVICE, [T][N] fp32, 16-byte aligned.  accumulate = 0 overwrites, 1 adds.
 *   workspace DEVICE scratch from afx_workspace_bytes(N, T), initialised once.
 */
afx_status afx_sparse_gemv(const void* Wt, int dtype, int K, int N, int64_t ldw, const void* x,
                           int T, const int32_t* idx, const int32_t* count, const int32_t* slot,
                           float* y, int accumulate, void* workspace, void* stream);

#ifdef __cplusplus
}
#endif
#endif /* AFX_H */
