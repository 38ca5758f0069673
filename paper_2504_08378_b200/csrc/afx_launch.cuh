// Host-side launch helpers: cluster occupancy table and tile-shape choice for the GEMV kernels.
#pragma once

#include <mutex>
#include <vector>

#include "afx_gemv.cuh"

namespace afx {

// Raises a kernel's dynamic shared-memory limit to at least `dyn_smem` (needed as soon as
// static + dynamic exceed 48 KB).  Remembers the largest value set per (device, kernel).
inline bool ensure_dyn_smem(const void* kern, size_t dyn_smem) {
    struct Entry {
        int dev;
        const void* kern;
        size_t smem;
    };
    static std::mutex mu;
    static std::vector<Entry> cache;
    if (dyn_smem == 0) return true;
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess) return false;
    std::lock_guard<std::mutex> lock(mu);
    for (Entry& e : cache)
        if (e.dev == dev && e.kern == kern) {
            if (e.smem >= dyn_smem) return true;
            if (cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                     static_cast<int>(dyn_smem)) != cudaSuccess)
                return false;
            e.smem = dyn_smem;
            return true;
        }
    if (cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize,
                             static_cast<int>(dyn_smem)) != cudaSuccess)
        return false;
    cache.push_back({dev, kern, dyn_smem});
    return true;
}

// How many clusters of S blocks of `kern` (`threads` threads, dyn_smem bytes of dynamic shared
// memory) the current device keeps resident at once.  Cached per (device, kernel, S,
// dyn_smem).  Returns 0 if the query fails.
inline int max_active_clusters(const void* kern, int S, size_t dyn_smem, int threads = kGemvThreads) {
    struct Entry {
        int dev;
        const void* kern;
        int S;
        size_t smem;
        int n;
    };
    static std::mutex mu;
    static std::vector<Entry> cache;
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess) return 0;
    std::lock_guard<std::mutex> lock(mu);
    for (const Entry& e : cache)
        if (e.dev == dev && e.kern == kern && e.S == S && e.smem == dyn_smem) return e.n;
    ensure_dyn_smem(kern, dyn_smem);
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3(S, 1, 1);
    cfg.blockDim = dim3(threads, 1, 1);
    cfg.dynamicSmemBytes = dyn_smem;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeClusterDimension;
    attr[0].val.clusterDim.x = S;
    attr[0].val.clusterDim.y = 1;
    attr[0].val.clusterDim.z = 1;
    cfg.attrs = attr;
    cfg.numAttrs = 1;
    int n = 0;
    if (cudaOccupancyMaxActiveClusters(&n, kern, &cfg) != cudaSuccess) {
        cudaGetLastError();
        n = 0;
    }
    cache.push_back({dev, kern, S, dyn_smem, n});
    return n;
}

// Where the device rows of a host-resident operator live (for the layer step over such operators).
struct HostedRows {
    const void* rows;
    int64_t ldw;
    int K, N;
};
HostedRows cache_rows(const afx_cache* cache);  // afx_cache.cu
HostedRows swap_rows(const afx_swap* swap);     // afx_swap.cu (rows = NULL: afx_swap_acquire returns them per layer)

struct GemvShapeChoice {
    int pw;     // tile width: 256, 128 or 64 outputs
    int S;      // blocks per cluster (= per tile)
    int tiles;  // ceil(N / pw)
};

// Widest tile and largest cluster such that all tiles' clusters are resident at once
// (one wave) and the block count is as large as possible.  kerns[i] is the kernel
// instantiated for tile width widest >> i.
#ifdef AFX_EXPERIMENT
extern int g_force_pw, g_force_s;  // experiment knobs (0 = automatic)
extern int g_cluster_margin;      // experiment knob (< 0 = automatic)
#endif

inline GemvShapeChoice choose_gemv_shape(int N, const void* const kerns[3], size_t dyn_smem,
                                         int extra_clusters = 0, int widest = 256, int groups = 1) {
#ifdef AFX_EXPERIMENT
    const int force_pw = g_force_pw, force_s = g_force_s, force_margin = g_cluster_margin;
#else
    constexpr int force_pw = 0, force_s = 0, force_margin = -1;
#endif
    GemvShapeChoice best = {widest >> 2, 1, groups * ((N + (widest >> 2) - 1) / (widest >> 2))};
    int best_blocks = -1;
    for (int i = 0; i < 3; ++i) {
        const int pw = widest >> i;
        if (force_pw && pw != force_pw) continue;
        const int tiles = groups * ((N + pw - 1) / pw);  // (groups operators of N outputs side by side)
        int s_fit = 0;
        for (int S = kMaxCluster; S >= 1; --S) {
            if (force_s && S != force_s) continue;
            // The occupancy query counts free block slots per GPC; launched behind another
            // kernel, two clusters fewer than it reports were seen resident at once (the
            // last ones then ran as a second wave), so a margin stays free.
            const int margin = force_margin >= 0 ? force_margin : (tiles + 15) / 16 < 2 ? 2 : (tiles + 15) / 16;
            if (max_active_clusters(kerns[i], S, dyn_smem) >= tiles + extra_clusters + margin) {
                s_fit = S;
                break;
            }
        }
        const int S = s_fit > 0 ? s_fit : (force_s ? force_s : 1);
        const int blocks = s_fit > 0 ? tiles * S : 0;  // 0: does not fit in one wave
        if (blocks > best_blocks) {
            best_blocks = blocks;
            best = {pw, S, tiles};
        }
    }
    return best;
}

// Launch `kern` on a (S, tiles) grid of S-block clusters, as a programmatic dependent of
// the work already in the stream.
template <class Kern, class Args>
inline afx_status launch_clustered(Kern kern, int S, int tiles, size_t dyn_smem, const Args& a,
                                   cudaStream_t st, int threads = kGemvThreads) {
    if (!ensure_dyn_smem(reinterpret_cast<const void*>(kern), dyn_smem)) {
        cudaGetLastError();
        return AFX_ERR_CUDA;
    }
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3(S, tiles, 1);
    cfg.blockDim = dim3(threads, 1, 1);
    cfg.dynamicSmemBytes = dyn_smem;
    cfg.stream = st;
    cudaLaunchAttribute attr[2];
    attr[0].id = cudaLaunchAttributeClusterDimension;
    attr[0].val.clusterDim.x = S;
    attr[0].val.clusterDim.y = 1;
    attr[0].val.clusterDim.z = 1;
    attr[1].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[1].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr;
    cfg.numAttrs = 2;
    return cudaLaunchKernelEx(&cfg, kern, a) == cudaSuccess ? AFX_OK : AFX_ERR_CUDA;
}

}  // namespace afx
