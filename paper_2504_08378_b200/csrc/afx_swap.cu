// afx_swap_*: cross-layer-group weight swapping of one operator type whose weights live in
// host memory (Sec. 3 "Cross-layer Active Weight Preloading" and its data layout; Sec. 4:
// operations PL "preload" and L "on-demand load" of the swapping pipeline).
//
// Host image: groups of d consecutive layers; inside a group the columns are ordered by
// channel id, then layer id, so the d columns a predicted channel needs in the d layers of a
// group are ONE contiguous chunk.  Device: two buffers (groups alternate between them), each
// [d][rows_pred + rows_miss][ldw]; layer i of the group reads rows [i][*] through
// afx_sparse_gemv's slot list.  The preload runs on a loader stream, ordered against the
// compute stream by events (the paper's request / complete signals): it starts once the
// predicting list exists and the compute stream waits for it at the group's first acquire.
#include <string.h>

#include <new>

#include "afx_launch.cuh"
#include "afx_select.cuh"

namespace afx {

constexpr int kSwapCopyThreads = 256;
constexpr int kSwapPolicyThreads = 1024;

struct SwapDev {
    int K, N, d, L, rows_pred, rows_miss;
    int64_t ldw16;            // row stride in 16-byte units
    const uint4* host;        // device view of the host image
    uint4* rows;              // [2][d][rows_pred + rows_miss][ldw16]
    int32_t* pred_slot;       // [2][K]: row of a preloaded channel, -1 otherwise
    int32_t* n_pred;          // [2]: channels preloaded into the buffer
    int32_t* fetch_ch;        // [K] on-demand channels of the last acquire
    int32_t* n_fetch;         // [1]
    int32_t* pred_list;       // [2][K + 1]: the object's own copy of a predicted list (count last)
};

__host__ __device__ inline int64_t swap_offset16(int L, int d, int K, int64_t ldw16, int layer, int channel) {
    const int g = layer / d, i = layer - g * d;
    const int dg = min(d, L - g * d);
    return (static_cast<int64_t>(g) * d * K + static_cast<int64_t>(channel) * dg + i) * ldw16;
}

__device__ __forceinline__ int64_t buffer_row16(const SwapDev& s, int buf, int layer_in_group, int row) {
    const int64_t per_layer = static_cast<int64_t>(s.rows_pred + s.rows_miss) * s.ldw16;
    return (static_cast<int64_t>(buf) * s.d + layer_in_group) * per_layer + static_cast<int64_t>(row) * s.ldw16;
}

__global__ void swap_clear_kernel(int32_t* pred_slot, int K, int32_t* n_pred) {
    for (int j = blockIdx.x * blockDim.x + threadIdx.x; j < K; j += gridDim.x * blockDim.x) pred_slot[j] = -1;
    if (blockIdx.x == 0 && threadIdx.x == 0) *n_pred = 0;
}

// Preload of group g into buffer buf: the c-th predicted channel (c < rows_pred) goes to row c
// of every layer of the group; its dg columns are one contiguous chunk of the host image.
__global__ void __launch_bounds__(kSwapCopyThreads)
swap_preload_kernel(SwapDev s, int g, int buf, const int32_t* __restrict__ idxP, const int32_t* __restrict__ cntP,
                    int32_t* __restrict__ status) {
    int n = *cntP;
    if (n < 0 || n > s.K) {
        if (blockIdx.x == 0 && threadIdx.x == 0) report_status(status, AFX_ERR_CAPACITY);
        n = max(0, min(n, s.K));
    }
    n = min(n, s.rows_pred);
    const int dg = min(s.d, s.L - g * s.d);
    const int n16 = s.N >> 3;
    int32_t* pred_slot = s.pred_slot + static_cast<size_t>(buf) * s.K;
    if (blockIdx.x == 0 && threadIdx.x == 0) s.n_pred[buf] = n;
    for (int c = blockIdx.x; c < n; c += gridDim.x) {
        const int j = idxP[c];
        if (static_cast<unsigned>(j) >= static_cast<unsigned>(s.K)) {
            if (threadIdx.x == 0) report_status(status, AFX_ERR_INVALID_ARG);
            continue;
        }
        if (threadIdx.x == 0) pred_slot[j] = c;
        const uint4* src = s.host + swap_offset16(s.L, s.d, s.K, s.ldw16, g * s.d, j);  // the chunk: dg rows of ldw16
        const int total = dg * n16;
        for (int e = threadIdx.x; e < total; e += 4 * kSwapCopyThreads) {
            uint4 v[4];
            int i[4], q[4];
#pragma unroll
            for (int u = 0; u < 4; ++u) {
                const int ee = e + u * kSwapCopyThreads;
                i[u] = ee / n16;
                q[u] = ee - i[u] * n16;
                if (ee < total) v[u] = src[static_cast<int64_t>(i[u]) * s.ldw16 + q[u]];
            }
#pragma unroll
            for (int u = 0; u < 4; ++u)
                if (e + u * kSwapCopyThreads < total) s.rows[buffer_row16(s, buf, i[u], c) + q[u]] = v[u];
        }
    }
}

// Where the channels of the actual active list are: preloaded row, or the next on-demand row.
__global__ void __launch_bounds__(kSwapPolicyThreads, 1)
swap_acquire_kernel(SwapDev s, int buf, const int32_t* __restrict__ idxA, const int32_t* __restrict__ cntA,
                    int32_t* __restrict__ slot_out, afx_swap_stats* __restrict__ stats, int32_t* __restrict__ status,
                    int dg) {
    __shared__ int scan[32];
    __shared__ int s_bad;
    int n = *cntA;
    if (n < 0 || n > s.K) {
        if (threadIdx.x == 0) report_status(status, AFX_ERR_CAPACITY);
        n = max(0, min(n, s.K));
    }
    if (threadIdx.x == 0) s_bad = 0;
    __syncthreads();
    const int32_t* pred_slot = s.pred_slot + static_cast<size_t>(buf) * s.K;
    const int per = (n + blockDim.x - 1) / blockDim.x;
    const int lo = min(static_cast<int>(threadIdx.x) * per, n), hi = min(lo + per, n);
    int mine = 0, bad = 0;
    for (int c = lo; c < hi; ++c) {
        const int j = idxA[c];
        const bool ok = static_cast<unsigned>(j) < static_cast<unsigned>(s.K);
        bad += !ok;
        mine += ok && pred_slot[j] < 0;
    }
    if (bad) atomicAdd(&s_bad, bad);
    int n_miss;
    int m = block_prefix(mine, scan, n_miss);
    for (int c = lo; c < hi; ++c) {
        const int j = idxA[c];
        int row = -1;
        if (static_cast<unsigned>(j) < static_cast<unsigned>(s.K)) {
            row = pred_slot[j];
            if (row < 0) {
                if (m < s.rows_miss) {
                    row = s.rows_pred + m;
                    s.fetch_ch[m] = j;
                }
                ++m;
            }
        }
        slot_out[c] = row;
    }
    __syncthreads();
    if (threadIdx.x == 0) {
        const int placed = min(n_miss, s.rows_miss);
        *s.n_fetch = placed;
        if (s_bad > 0) report_status(status, AFX_ERR_INVALID_ARG);
        if (n_miss > placed) report_status(status, AFX_ERR_CAPACITY);
        if (stats != nullptr) {
            stats->hits = n - n_miss - s_bad;
            stats->ondemand = placed;
            stats->overflow = n_miss - placed;
            stats->preloaded = s.n_pred[buf];
            stats->bytes_preload = static_cast<unsigned long long>(s.n_pred[buf]) * dg * s.N * 2ull;
            stats->bytes_ondemand = static_cast<unsigned long long>(placed) * s.N * 2ull;
        }
    }
}

// On-demand load: single columns of this layer.
__global__ void __launch_bounds__(kSwapCopyThreads)
swap_fetch_kernel(SwapDev s, int layer, int buf) {
    const int n = *s.n_fetch;
    const int n16 = s.N >> 3;
    const int i = layer % s.d;
    for (int f = blockIdx.x; f < n; f += gridDim.x) {
        const uint4* src = s.host + swap_offset16(s.L, s.d, s.K, s.ldw16, layer, s.fetch_ch[f]);
        uint4* dst = s.rows + buffer_row16(s, buf, i, s.rows_pred + f);
        for (int e = threadIdx.x; e < n16; e += 4 * kSwapCopyThreads) {
            uint4 v[4];
#pragma unroll
            for (int u = 0; u < 4; ++u)
                if (e + u * kSwapCopyThreads < n16) v[u] = src[e + u * kSwapCopyThreads];
#pragma unroll
            for (int u = 0; u < 4; ++u)
                if (e + u * kSwapCopyThreads < n16) dst[e + u * kSwapCopyThreads] = v[u];
        }
    }
}

}  // namespace afx

struct afx_swap {
    afx_swap_desc d;
    afx::SwapDev dev;
    void* arena = nullptr;
    cudaStream_t loader = nullptr;
    bool own_loader = false;
    cudaEvent_t ev_req[2] = {nullptr, nullptr}, ev_done[2] = {nullptr, nullptr};
    int group_in_buf[2] = {-1, -1};  // which group's preload the buffer holds (host bookkeeping)
    bool pending[2] = {false, false};  // a preload whose completion the compute stream has not waited for yet
    int n_groups = 0;
};

namespace afx {
HostedRows swap_rows(const afx_swap* swap) { return {nullptr, swap->d.ldw, swap->d.K, swap->d.N}; }
}  // namespace afx

extern "C" size_t afx_swap_host_offset(int n_layers, int group, int K, int64_t ldw, int layer, int channel) {
    if (n_layers < 1 || group < 1 || K < 1 || ldw < 1 || layer < 0 || layer >= n_layers || channel < 0 || channel >= K)
        return static_cast<size_t>(-1);
    const int g = layer / group, i = layer - g * group;
    const int dg = group < n_layers - g * group ? group : n_layers - g * group;
    return (static_cast<size_t>(g) * group * K + static_cast<size_t>(channel) * dg + i) * static_cast<size_t>(ldw);
}

extern "C" afx_status afx_swap_pack_host(const void* const* per_layer, int n_layers, int group, int K, int64_t ldw,
                                         void* host_out) {
    if (per_layer == nullptr || host_out == nullptr || n_layers < 1 || group < 1 || K < 1 || ldw < 1)
        return AFX_ERR_INVALID_ARG;
    const size_t row = static_cast<size_t>(ldw) * 2;
    for (int l = 0; l < n_layers; ++l) {
        if (per_layer[l] == nullptr) return AFX_ERR_INVALID_ARG;
        const char* src = static_cast<const char*>(per_layer[l]);
        for (int j = 0; j < K; ++j)
            memcpy(static_cast<char*>(host_out) + afx_swap_host_offset(n_layers, group, K, ldw, l, j) * 2, src + j * row, row);
    }
    return AFX_OK;
}

extern "C" size_t afx_swap_device_bytes(const afx_swap_desc* desc) {
    if (desc == nullptr || desc->group < 1 || desc->rows_pred < 0 || desc->rows_miss < 0 || desc->ldw < 1) return 0;
    return static_cast<size_t>(2) * desc->group * (static_cast<size_t>(desc->rows_pred) + desc->rows_miss) *
           static_cast<size_t>(desc->ldw) * 2;
}

extern "C" afx_status afx_swap_create(const afx_swap_desc* desc, afx_swap** out) {
    using namespace afx;
    if (desc == nullptr || out == nullptr) return AFX_ERR_INVALID_ARG;
    const afx_swap_desc& d = *desc;
    if (d.dtype != AFX_F16 && d.dtype != AFX_BF16) return AFX_ERR_UNSUPPORTED;
    if (d.n_layers < 1 || d.group < 1 || d.K < 1 || d.K > (1 << 20) || d.N < 1 || d.ldw < d.N || d.rows_pred < 0 ||
        d.rows_miss < 0 || d.rows_pred + d.rows_miss < 1 || d.host_base == nullptr || d.dev_rows == nullptr)
        return AFX_ERR_INVALID_ARG;
    if ((d.N & 7) != 0 || (d.ldw & 7) != 0 || !aligned16(d.host_base) || !aligned16(d.dev_rows)) return AFX_ERR_ALIGNMENT;
    void* host_dev = nullptr;
    if (cudaHostGetDevicePointer(&host_dev, const_cast<void*>(d.host_base), 0) != cudaSuccess || host_dev == nullptr) {
        cudaGetLastError();
        return AFX_ERR_INVALID_ARG;  // not page-locked / not mapped
    }
    afx_swap* s = new (std::nothrow) afx_swap();
    if (s == nullptr) return AFX_ERR_CAPACITY;
    s->d = d;
    s->n_groups = (d.n_layers + d.group - 1) / d.group;
    const size_t K = static_cast<size_t>(d.K);
    auto up = [](size_t b) { return (b + 255) / 256 * 256; };
    const size_t o_pred = 0, o_np = o_pred + up(2 * K * 4), o_fch = o_np + 256, o_nf = o_fch + up(K * 4),
                 o_pl = o_nf + 256, total = o_pl + up(2 * (K + 1) * 4);
    char* arena = nullptr;
    bool ok = cudaMalloc(reinterpret_cast<void**>(&arena), total) == cudaSuccess;
    ok = ok && cudaMemset(arena, 0xFF, up(2 * K * 4)) == cudaSuccess && cudaMemset(arena + o_np, 0, total - o_np) == cudaSuccess;
    if (ok && d.loader_stream == nullptr) {
        ok = cudaStreamCreateWithFlags(&s->loader, cudaStreamNonBlocking) == cudaSuccess;
        s->own_loader = ok;
    } else {
        s->loader = static_cast<cudaStream_t>(d.loader_stream);
    }
    for (int b = 0; ok && b < 2; ++b)
        ok = cudaEventCreateWithFlags(&s->ev_req[b], cudaEventDisableTiming) == cudaSuccess &&
             cudaEventCreateWithFlags(&s->ev_done[b], cudaEventDisableTiming) == cudaSuccess;
    if (!ok) {
        cudaGetLastError();
        s->arena = arena;
        afx_swap_destroy(s);
        return AFX_ERR_CUDA;
    }
    s->arena = arena;
    SwapDev& v = s->dev;
    v.K = d.K;
    v.N = d.N;
    v.d = d.group;
    v.L = d.n_layers;
    v.rows_pred = d.rows_pred;
    v.rows_miss = d.rows_miss;
    v.ldw16 = d.ldw / 8;
    v.host = static_cast<const uint4*>(host_dev);
    v.rows = static_cast<uint4*>(d.dev_rows);
    v.pred_slot = reinterpret_cast<int32_t*>(arena + o_pred);
    v.n_pred = reinterpret_cast<int32_t*>(arena + o_np);
    v.fetch_ch = reinterpret_cast<int32_t*>(arena + o_fch);
    v.n_fetch = reinterpret_cast<int32_t*>(arena + o_nf);
    v.pred_list = reinterpret_cast<int32_t*>(arena + o_pl);
    *out = s;
    return AFX_OK;
}

extern "C" afx_status afx_swap_destroy(afx_swap* s) {
    if (s == nullptr) return AFX_ERR_INVALID_ARG;
    for (int b = 0; b < 2; ++b) {
        if (s->ev_req[b] != nullptr) cudaEventDestroy(s->ev_req[b]);
        if (s->ev_done[b] != nullptr) cudaEventDestroy(s->ev_done[b]);
    }
    if (s->own_loader && s->loader != nullptr) cudaStreamDestroy(s->loader);
    if (s->arena != nullptr) cudaFree(s->arena);
    delete s;
    return AFX_OK;
}

extern "C" afx_status afx_swap_preload(afx_swap* s, int group_index, const int32_t* idxP, const int32_t* cntP,
                                       int copy_blocks, int32_t* dev_status, void* compute_stream) {
    using namespace afx;
    if (s == nullptr || idxP == nullptr || cntP == nullptr) return AFX_ERR_INVALID_ARG;
    if (group_index < 0 || group_index >= s->n_groups || copy_blocks < 0) return AFX_ERR_INVALID_ARG;
    if ((reinterpret_cast<uintptr_t>(idxP) & 3u) || (reinterpret_cast<uintptr_t>(cntP) & 3u) ||
        (reinterpret_cast<uintptr_t>(dev_status) & 3u))
        return AFX_ERR_ALIGNMENT;
    const int b = group_index & 1;
    cudaStream_t cs = static_cast<cudaStream_t>(compute_stream);
    const int blocks = copy_blocks > 0 ? copy_blocks : 32;
    // The caller's list may be overwritten by the next layer while the loader still reads it:
    // take a copy on the compute stream first.
    int32_t* own = s->dev.pred_list + static_cast<size_t>(b) * (s->dev.K + 1);
    if (cudaMemcpyAsync(own, idxP, static_cast<size_t>(s->dev.K) * 4, cudaMemcpyDeviceToDevice, cs) != cudaSuccess ||
        cudaMemcpyAsync(own + s->dev.K, cntP, 4, cudaMemcpyDeviceToDevice, cs) != cudaSuccess)
        return AFX_ERR_CUDA;
    // request: the list exists, and everything that still reads this buffer has been enqueued
    if (cudaEventRecord(s->ev_req[b], cs) != cudaSuccess || cudaStreamWaitEvent(s->loader, s->ev_req[b], 0) != cudaSuccess)
        return AFX_ERR_CUDA;
    swap_clear_kernel<<<8, 256, 0, s->loader>>>(s->dev.pred_slot + static_cast<size_t>(b) * s->dev.K, s->dev.K,
                                                 s->dev.n_pred + b);
    swap_preload_kernel<<<blocks, kSwapCopyThreads, 0, s->loader>>>(s->dev, group_index, b, own, own + s->dev.K, dev_status);
    if (cudaGetLastError() != cudaSuccess) return AFX_ERR_CUDA;
    // complete
    if (cudaEventRecord(s->ev_done[b], s->loader) != cudaSuccess) return AFX_ERR_CUDA;
    s->group_in_buf[b] = group_index;
    s->pending[b] = true;
    return AFX_OK;
}

extern "C" afx_status afx_swap_acquire(afx_swap* s, int layer, const int32_t* idxA, const int32_t* cntA,
                                       int32_t* slot_out, afx_swap_stats* stats, int32_t* dev_status,
                                       void* compute_stream, const void** rows_out) {
    using namespace afx;
    if (s == nullptr || idxA == nullptr || cntA == nullptr || slot_out == nullptr || rows_out == nullptr)
        return AFX_ERR_INVALID_ARG;
    if (layer < 0 || layer >= s->d.n_layers) return AFX_ERR_INVALID_ARG;
    if ((reinterpret_cast<uintptr_t>(idxA) & 3u) || (reinterpret_cast<uintptr_t>(cntA) & 3u) ||
        (reinterpret_cast<uintptr_t>(slot_out) & 3u) || (reinterpret_cast<uintptr_t>(stats) & 7u) ||
        (reinterpret_cast<uintptr_t>(dev_status) & 3u))
        return AFX_ERR_ALIGNMENT;
    const int g = layer / s->d.group, b = g & 1;
    cudaStream_t cs = static_cast<cudaStream_t>(compute_stream);
    if (s->group_in_buf[b] == g) {
        if (s->pending[b]) {  // first use of the group: wait for its preload
            if (cudaStreamWaitEvent(cs, s->ev_done[b], 0) != cudaSuccess) return AFX_ERR_CUDA;
            s->pending[b] = false;
        }
    } else {
        // nothing was preloaded for this group (the first group of a token, or a caller that does
        // not predict): an earlier preload into this buffer, if any, must be over before the
        // buffer is declared empty
        if (s->pending[b]) {
            if (cudaStreamWaitEvent(cs, s->ev_done[b], 0) != cudaSuccess) return AFX_ERR_CUDA;
            s->pending[b] = false;
        }
        swap_clear_kernel<<<8, 256, 0, cs>>>(s->dev.pred_slot + static_cast<size_t>(b) * s->dev.K, s->dev.K,
                                             s->dev.n_pred + b);
        s->group_in_buf[b] = g;
    }
    const int dg = s->d.group < s->d.n_layers - g * s->d.group ? s->d.group : s->d.n_layers - g * s->d.group;
    swap_acquire_kernel<<<1, kSwapPolicyThreads, 0, cs>>>(s->dev, b, idxA, cntA, slot_out, stats, dev_status, dg);
    const int blocks = 2 * (sm_count() > 0 ? sm_count() : 148);
    swap_fetch_kernel<<<blocks, kSwapCopyThreads, 0, cs>>>(s->dev, layer, b);
    const size_t per_layer = (static_cast<size_t>(s->d.rows_pred) + s->d.rows_miss) * static_cast<size_t>(s->d.ldw) * 2;
    *rows_out = static_cast<const char*>(s->d.dev_rows) + (static_cast<size_t>(b) * s->d.group + layer % s->d.group) * per_layer;
    return launch_status();
}
