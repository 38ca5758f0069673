// afx_cache_*: least-frequently-used column cache of one host-resident operator.
//
// The policy of one step runs in ONE thread block (it is integer bookkeeping over at most K
// channels; what costs time in a step is the host -> device copy of the misses): usage
// counts and an activity bitmap, ordered compactions (hits/misses in list order, free slots
// ascending), a bitonic sort of the eviction candidates by (count, channel id), a short
// sequential pass that pairs misses with candidates exactly as the step-by-step definition
// does, and the table updates.  A second kernel copies the missed columns from the mapped
// host memory with 128-bit loads.
#include <new>
#include <vector>

#include "afx_launch.cuh"
#include "afx_select.cuh"

namespace afx {

constexpr int kCacheThreads = 1024;
constexpr int kCopyThreads = 256;
constexpr int kCacheMaxK = 1 << 20;
constexpr unsigned long long kKeyPad = ~0ull;

struct CacheTables {
    int K, C, staging_rows;
    int32_t* slot_of;   // [K]
    int32_t* chan_of;   // [C]
    uint32_t* usage;    // [K]
    int32_t* miss_pos;  // [K] list positions of this step's misses, ascending
    int32_t* free_list; // [C]
    int32_t* fetch_ch;  // [K] channel to copy for miss i
    int32_t* fetch_row; // [K] destination row (-1: none)
    int32_t* n_fetch;   // [1]
    unsigned long long* keys;  // [P] sort area when it does not fit into shared memory
    int P;                     // power of two >= C
    int keys_in_smem;
};

// Ordered compaction helper: every thread owns the contiguous range [lo, hi) of n items.
__device__ __forceinline__ void owned_range(int n, int& lo, int& hi) {
    const int per = (n + blockDim.x - 1) / blockDim.x;
    lo = min(static_cast<int>(threadIdx.x) * per, n);
    hi = min(lo + per, n);
}

__global__ void __launch_bounds__(kCacheThreads, 1)
cache_policy_kernel(CacheTables tb, const int32_t* __restrict__ idx, const int32_t* __restrict__ count,
                    int32_t* __restrict__ slot_out, afx_cache_stats* __restrict__ stats, int N,
                    int32_t* __restrict__ status) {
    extern __shared__ __align__(16) unsigned char dyn[];
    __shared__ int scan[4][32];
    __shared__ int s_mfreq[kCacheThreads];
    __shared__ int s_assign[kCacheThreads];
    __shared__ int s_vp, s_nt, s_bad;
    const int K = tb.K, C = tb.C;
    const int nwords = (K + 31) >> 5;
    uint32_t* active = reinterpret_cast<uint32_t*>(dyn);
    unsigned long long* keys = tb.keys_in_smem
                                   ? reinterpret_cast<unsigned long long*>(dyn + (static_cast<size_t>(nwords) * 4 + 15) / 16 * 16)
                                   : tb.keys;
    const int tid = threadIdx.x;
    int n = *count;
    if (n < 0 || n > K) {
        if (tid == 0) report_status(status, AFX_ERR_CAPACITY);
        n = max(0, min(n, K));
    }
    // a list entry outside [0, K) takes no part in the step: no count, no slot (-1), neither a
    // hit nor a miss; the status word reports it
    auto valid = [&](int j) { return static_cast<unsigned>(j) < static_cast<unsigned>(K); };

    // 1. activity bitmap and usage counts
    for (int w = tid; w < nwords; w += blockDim.x) active[w] = 0u;
    if (tid == 0) {
        s_vp = 0;
        s_nt = 0;
        s_bad = 0;
    }
    __syncthreads();
    for (int c = tid; c < n; c += blockDim.x) {
        const int j = idx[c];
        if (!valid(j)) {
            atomicAdd(&s_bad, 1);
            continue;
        }
        atomicOr(&active[j >> 5], 1u << (j & 31));
        tb.usage[j] += 1u;  // list entries are distinct channels
    }
    __syncthreads();

    // 2. hits get their slot; misses are listed in list order
    int lo, hi;
    owned_range(n, lo, hi);
    int mine = 0;
    for (int c = lo; c < hi; ++c) mine += valid(idx[c]) && tb.slot_of[idx[c]] < 0;
    int n_miss;
    int at = block_prefix(mine, scan[0], n_miss);
    for (int c = lo; c < hi; ++c) {
        const int j = idx[c];
        const int s = valid(j) ? tb.slot_of[j] : -1;
        if (valid(j) && s < 0)
            tb.miss_pos[at++] = c;
        else
            slot_out[c] = s;
    }

    // 3. free slots ascending; 4. eviction candidates: cached channels not active in this step
    owned_range(C, lo, hi);
    int nf = 0, nv = 0;
    for (int s = lo; s < hi; ++s) {
        const int v = tb.chan_of[s];
        nf += v < 0;
        nv += v >= 0 && ((active[v >> 5] >> (v & 31)) & 1u) == 0u;
    }
    int n_free, n_cand;
    int fat = block_prefix(nf, scan[1], n_free);
    int vat = block_prefix(nv, scan[2], n_cand);
    int P = 1;
    while (P < n_cand) P <<= 1;
    const bool need_victims = n_miss > n_free && n_cand > 0;
    for (int s = lo; s < hi; ++s) {
        const int v = tb.chan_of[s];
        if (v < 0)
            tb.free_list[fat++] = s;
        else if (need_victims && ((active[v >> 5] >> (v & 31)) & 1u) == 0u)
            keys[vat++] = (static_cast<unsigned long long>(tb.usage[v]) << 32) | static_cast<uint32_t>(v);
    }
    if (need_victims)
        for (int i = n_cand + tid; i < P; i += blockDim.x) keys[i] = kKeyPad;
    __syncthreads();

    // 5. candidates ascending by (count, channel id)
    if (need_victims) {
        for (int k = 2; k <= P; k <<= 1) {
            for (int j = k >> 1; j > 0; j >>= 1) {
                for (int i = tid; i < P; i += blockDim.x) {
                    const int p = i ^ j;
                    if (p > i) {
                        const unsigned long long a = keys[i], b = keys[p];
                        const bool up = (i & k) == 0;
                        if ((a > b) == up) {
                            keys[i] = b;
                            keys[p] = a;
                        }
                    }
                }
                __syncthreads();
            }
        }
    }

    // 6./7. misses in ascending order: free slots first, then the candidates in order, a miss
    // taking the next candidate only when its count is not smaller; in chunks of blockDim.x
    for (int base = 0; base < n_miss; base += blockDim.x) {
        const int i = base + tid;
        int c = -1, j = -1;
        if (i < n_miss) {
            c = tb.miss_pos[i];
            j = idx[c];
            s_mfreq[tid] = static_cast<int>(tb.usage[j]);
        }
        __syncthreads();
        if (tid == 0) {
            int vp = s_vp, nt = s_nt;
            const int m = min(static_cast<int>(blockDim.x), n_miss - base);
            for (int q = 0; q < m; ++q) {
                if (base + q < n_free) {
                    s_assign[q] = 0;  // takes free_list[base + q]
                } else if (vp < n_cand && static_cast<uint32_t>(s_mfreq[q]) >= static_cast<uint32_t>(keys[vp] >> 32)) {
                    s_assign[q] = vp++;
                } else {
                    s_assign[q] = -1 - nt++;
                }
            }
            s_vp = vp;
            s_nt = nt;
        }
        __syncthreads();
        if (i < n_miss) {
            int row;
            const int a = s_assign[tid];
            if (i < n_free) {
                row = tb.free_list[i];
            } else if (a >= 0) {
                const int v = static_cast<int>(keys[a] & 0xFFFFFFFFull);
                row = tb.slot_of[v];
                tb.slot_of[v] = -1;
            } else {
                const int r = -1 - a;
                row = r < tb.staging_rows ? C + r : -1;
            }
            if (row >= 0 && row < C) {
                tb.chan_of[row] = j;
                tb.slot_of[j] = row;
            }
            slot_out[c] = row;
            tb.fetch_ch[i] = j;
            tb.fetch_row[i] = row;
        }
        __syncthreads();  // s_mfreq / s_assign are reused by the next chunk
    }
    if (tid == 0) {
        *tb.n_fetch = n_miss;
        const int nt = s_nt;
        const int over = max(0, nt - tb.staging_rows);
        if (s_bad > 0) report_status(status, AFX_ERR_INVALID_ARG);
        if (over > 0) report_status(status, AFX_ERR_CAPACITY);
        if (stats != nullptr) {
            stats->hits = n - n_miss - s_bad;
            stats->misses = n_miss;
            stats->transients = nt;
            stats->overflow = over;
            stats->bytes_fetched = static_cast<unsigned long long>(n_miss - over) * static_cast<unsigned long long>(N) * 2ull;
        }
    }
}

// Copies fetch_ch[f] -> row fetch_row[f] for f < *n_fetch; one column per block at a time.
__global__ void __launch_bounds__(kCopyThreads)
cache_copy_kernel(const uint4* __restrict__ host, uint4* __restrict__ slots, int64_t ldw16, int n16,
                  const int32_t* __restrict__ fetch_ch, const int32_t* __restrict__ fetch_row,
                  const int32_t* __restrict__ n_fetch) {
    const int n = *n_fetch;
    for (int f = blockIdx.x; f < n; f += gridDim.x) {
        const int row = fetch_row[f];
        if (row < 0) continue;
        const uint4* src = host + static_cast<int64_t>(fetch_ch[f]) * ldw16;
        uint4* dst = slots + static_cast<int64_t>(row) * ldw16;
        for (int i = threadIdx.x; i < n16; i += 4 * kCopyThreads) {
            uint4 v[4];
#pragma unroll
            for (int u = 0; u < 4; ++u)
                if (i + u * kCopyThreads < n16) v[u] = src[i + u * kCopyThreads];
#pragma unroll
            for (int u = 0; u < 4; ++u)
                if (i + u * kCopyThreads < n16) dst[i + u * kCopyThreads] = v[u];
        }
    }
}

}  // namespace afx

struct afx_cache {
    afx_cache_desc d;
    afx::CacheTables tb;
    const void* host_dev;  // device view of host_base
    size_t policy_smem;
    void* arena;           // one cudaMalloc holding every table
};

namespace afx {
HostedRows cache_rows(const afx_cache* cache) { return {cache->d.slots, cache->d.ldw, cache->d.K, cache->d.N}; }
}  // namespace afx

extern "C" afx_status afx_cache_create(const afx_cache_desc* desc, afx_cache** out) {
    using namespace afx;
    if (desc == nullptr || out == nullptr) return AFX_ERR_INVALID_ARG;
    const afx_cache_desc& d = *desc;
    if (d.dtype != AFX_F16 && d.dtype != AFX_BF16) return AFX_ERR_UNSUPPORTED;
    if (d.K < 1 || d.K > kCacheMaxK || d.N < 1 || d.ldw < d.N || d.staging_rows < 0 || d.host_base == nullptr ||
        d.slots == nullptr)
        return AFX_ERR_INVALID_ARG;
    if (d.capacity < 1 || d.capacity > d.K) return AFX_ERR_CAPACITY;
    if ((d.N & 7) != 0 || (d.ldw & 7) != 0 || !aligned16(d.host_base) || !aligned16(d.slots)) return AFX_ERR_ALIGNMENT;
    void* host_dev = nullptr;
    if (cudaHostGetDevicePointer(&host_dev, const_cast<void*>(d.host_base), 0) != cudaSuccess || host_dev == nullptr) {
        cudaGetLastError();
        return AFX_ERR_INVALID_ARG;  // not page-locked / not mapped
    }
    afx_cache* c = new (std::nothrow) afx_cache();
    if (c == nullptr) return AFX_ERR_CAPACITY;
    c->d = d;
    c->host_dev = host_dev;
    int P = 1;
    while (P < d.capacity) P <<= 1;
    const size_t K = static_cast<size_t>(d.K), C = static_cast<size_t>(d.capacity);
    auto up = [](size_t b) { return (b + 255) / 256 * 256; };
    const size_t o_slot = 0, o_chan = o_slot + up(K * 4), o_use = o_chan + up(C * 4), o_miss = o_use + up(K * 4),
                 o_free = o_miss + up(K * 4), o_fch = o_free + up(C * 4), o_frow = o_fch + up(K * 4),
                 o_nf = o_frow + up(K * 4), o_keys = o_nf + 256, total = o_keys + up(static_cast<size_t>(P) * 8);
    char* arena = nullptr;
    if (cudaMalloc(reinterpret_cast<void**>(&arena), total) != cudaSuccess) {
        cudaGetLastError();
        delete c;
        return AFX_ERR_CUDA;
    }
    c->arena = arena;
    CacheTables& tb = c->tb;
    tb.K = d.K;
    tb.C = d.capacity;
    tb.staging_rows = d.staging_rows;
    tb.slot_of = reinterpret_cast<int32_t*>(arena + o_slot);
    tb.chan_of = reinterpret_cast<int32_t*>(arena + o_chan);
    tb.usage = reinterpret_cast<uint32_t*>(arena + o_use);
    tb.miss_pos = reinterpret_cast<int32_t*>(arena + o_miss);
    tb.free_list = reinterpret_cast<int32_t*>(arena + o_free);
    tb.fetch_ch = reinterpret_cast<int32_t*>(arena + o_fch);
    tb.fetch_row = reinterpret_cast<int32_t*>(arena + o_frow);
    tb.n_fetch = reinterpret_cast<int32_t*>(arena + o_nf);
    tb.keys = reinterpret_cast<unsigned long long*>(arena + o_keys);
    tb.P = P;
    const size_t bitmap = (static_cast<size_t>((d.K + 31) >> 5) * 4 + 15) / 16 * 16;
    tb.keys_in_smem = bitmap + static_cast<size_t>(P) * 8 <= 192 * 1024;
    c->policy_smem = bitmap + (tb.keys_in_smem ? static_cast<size_t>(P) * 8 : 0);
    // empty cache: no channel has a slot, no slot has a channel, all counts zero
    if (cudaMemset(tb.slot_of, 0xFF, K * 4) != cudaSuccess || cudaMemset(tb.chan_of, 0xFF, C * 4) != cudaSuccess ||
        cudaMemset(tb.usage, 0, K * 4) != cudaSuccess || cudaMemset(tb.n_fetch, 0, 4) != cudaSuccess ||
        !ensure_dyn_smem(reinterpret_cast<const void*>(cache_policy_kernel), c->policy_smem)) {
        cudaGetLastError();
        cudaFree(arena);
        delete c;
        return AFX_ERR_CUDA;
    }
    *out = c;
    return AFX_OK;
}

extern "C" afx_status afx_cache_destroy(afx_cache* cache) {
    if (cache == nullptr) return AFX_ERR_INVALID_ARG;
    if (cache->arena != nullptr) cudaFree(cache->arena);
    delete cache;
    return AFX_OK;
}

extern "C" afx_status afx_cache_reset(afx_cache* cache, void* stream) {
    if (cache == nullptr) return AFX_ERR_INVALID_ARG;
    return cudaMemsetAsync(cache->tb.usage, 0, static_cast<size_t>(cache->tb.K) * 4,
                           static_cast<cudaStream_t>(stream)) == cudaSuccess
               ? AFX_OK
               : AFX_ERR_CUDA;
}

extern "C" afx_status afx_cache_install(afx_cache* cache, const int32_t* host_channels, int n, void* stream) {
    if (cache == nullptr || (n > 0 && host_channels == nullptr) || n < 0) return AFX_ERR_INVALID_ARG;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    const afx::CacheTables& tb = cache->tb;
    std::vector<int32_t> slot_of(tb.K), chan_of(tb.C);
    if (cudaMemcpyAsync(slot_of.data(), tb.slot_of, slot_of.size() * 4, cudaMemcpyDeviceToHost, st) != cudaSuccess ||
        cudaMemcpyAsync(chan_of.data(), tb.chan_of, chan_of.size() * 4, cudaMemcpyDeviceToHost, st) != cudaSuccess ||
        cudaStreamSynchronize(st) != cudaSuccess)
        return AFX_ERR_CUDA;
    int next = 0;
    const size_t row_bytes = static_cast<size_t>(cache->d.N) * 2, stride = static_cast<size_t>(cache->d.ldw) * 2;
    for (int i = 0; i < n; ++i) {
        const int j = host_channels[i];
        if (j < 0 || j >= tb.K || slot_of[j] >= 0) return AFX_ERR_INVALID_ARG;
        while (next < tb.C && chan_of[next] >= 0) ++next;
        if (next >= tb.C) return AFX_ERR_CAPACITY;
        chan_of[next] = j;
        slot_of[j] = next;
        if (cudaMemcpyAsync(static_cast<char*>(cache->d.slots) + next * stride,
                            static_cast<const char*>(cache->d.host_base) + j * stride, row_bytes,
                            cudaMemcpyHostToDevice, st) != cudaSuccess)
            return AFX_ERR_CUDA;
    }
    if (cudaMemcpyAsync(tb.slot_of, slot_of.data(), slot_of.size() * 4, cudaMemcpyHostToDevice, st) != cudaSuccess ||
        cudaMemcpyAsync(tb.chan_of, chan_of.data(), chan_of.size() * 4, cudaMemcpyHostToDevice, st) != cudaSuccess ||
        cudaStreamSynchronize(st) != cudaSuccess)
        return AFX_ERR_CUDA;
    return AFX_OK;
}

extern "C" afx_status afx_cache_fetch(afx_cache* cache, const int32_t* idx, const int32_t* count, int32_t* slot_out,
                                      afx_cache_stats* stats, int32_t* dev_status, void* stream) {
    using namespace afx;
    if (cache == nullptr || idx == nullptr || count == nullptr || slot_out == nullptr) return AFX_ERR_INVALID_ARG;
    if ((reinterpret_cast<uintptr_t>(idx) & 3u) || (reinterpret_cast<uintptr_t>(count) & 3u) ||
        (reinterpret_cast<uintptr_t>(slot_out) & 3u) || (reinterpret_cast<uintptr_t>(stats) & 7u) ||
        (reinterpret_cast<uintptr_t>(dev_status) & 3u))
        return AFX_ERR_ALIGNMENT;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    cache_policy_kernel<<<1, kCacheThreads, cache->policy_smem, st>>>(cache->tb, idx, count, slot_out, stats,
                                                                       cache->d.N, dev_status);
    if (cudaGetLastError() != cudaSuccess) return AFX_ERR_CUDA;
    const int blocks = 4 * (sm_count() > 0 ? sm_count() : 148);
    cache_copy_kernel<<<blocks, kCopyThreads, 0, st>>>(
        static_cast<const uint4*>(cache->host_dev), static_cast<uint4*>(cache->d.slots), cache->d.ldw / 8,
        cache->d.N / 8, cache->tb.fetch_ch, cache->tb.fetch_row, cache->tb.n_fetch);
    return launch_status();
}

extern "C" afx_status afx_cache_snapshot(afx_cache* cache, int32_t* host_slot_of, uint32_t* host_usage, void* stream) {
    if (cache == nullptr) return AFX_ERR_INVALID_ARG;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    const size_t bytes = static_cast<size_t>(cache->tb.K) * 4;
    if (host_slot_of != nullptr &&
        cudaMemcpyAsync(host_slot_of, cache->tb.slot_of, bytes, cudaMemcpyDeviceToHost, st) != cudaSuccess)
        return AFX_ERR_CUDA;
    if (host_usage != nullptr &&
        cudaMemcpyAsync(host_usage, cache->tb.usage, bytes, cudaMemcpyDeviceToHost, st) != cudaSuccess)
        return AFX_ERR_CUDA;
    return cudaStreamSynchronize(st) == cudaSuccess ? AFX_OK : AFX_ERR_CUDA;
}
