// afx_select_active / afx_diff_active: stand-alone selection and cross-layer set difference.
#include "afx_launch.cuh"
#include "afx_select.cuh"

namespace afx {

constexpr int kSelectThreads = 1024;

// Dynamic shared memory.  Fast path: [flag words, padded to 16 bytes] [one token's keys] [key
// histogram].  Large-K path: flag words only.
static size_t select_dyn_smem(int K) {
    size_t b = (static_cast<size_t>((K + 31) >> 5) * 4 + 15) / 16 * 16;
    if (K <= kSelectFastMaxK) b += (static_cast<size_t>(K) + 7) / 8 * 8 * 2 + kKeyHistBytes;
    return b;
}

template <int DT>
__global__ void __launch_bounds__(kSelectThreads, 1)
select_kernel(const uint16_t* __restrict__ x, int K, int T, int mode, int k, float tau,
              int32_t* __restrict__ idx, int32_t* __restrict__ count, uint32_t* __restrict__ bitmap) {
    extern __shared__ __align__(16) unsigned char s_dyn[];
    __shared__ SelectScratch scratch;
    const int nwords = (K + 31) >> 5;
    const size_t flag_bytes = (static_cast<size_t>(nwords) * 4 + 15) / 16 * 16;
    uint32_t* s_flags = reinterpret_cast<uint32_t*>(s_dyn);
    const int lane = lane_id();
    if (K <= kSelectFastMaxK) {
        uint16_t* xs = reinterpret_cast<uint16_t*>(s_dyn + flag_bytes);
        uint32_t* hist = reinterpret_cast<uint32_t*>(s_dyn + flag_bytes + (static_cast<size_t>(K) + 7) / 8 * 8 * 2);
        const bool topk = mode == AFX_MODE_TOPK && k > 0 && k < K;
        if (topk) block_clear_key_hist<kSelectThreads>(hist);
        unsigned long long fl = 0ull;
        int pos0 = 0, total = 0;
        for (int t = 0; t < T; ++t) {
            if (t > 0) __syncthreads();  // the previous token's keys are still being read
            block_stage_token(x + static_cast<size_t>(t) * K, K, xs);
            fl |= block_token_flags<DT, kSelectThreads>(xs, K, mode, k, tau, hist, t == 0, &scratch, T == 1,
                                                        pos0, total);
        }
        if (T > 1) pos0 = block_prefix(__popcll(fl), scratch.wtot[2], total);
        for_each_owned_active(fl, K, pos0, [&](int j, int pos) { idx[pos] = j; });
        if (threadIdx.x == 0) *count = total;
        if (bitmap != nullptr) {
            store_flag_bytes(fl, K, s_flags);
            __syncthreads();
            for (int w = threadIdx.x; w < nwords; w += blockDim.x) bitmap[w] = s_flags[w];
        }
        return;
    }
    int w0, w1;
    warp_word_range(nwords, w0, w1);
    int mine = 0;
    block_select_flags_large<DT>(x, K, T, mode, k, tau, s_flags, &scratch);
    for (int w = w0 + lane; w < w1; w += 32) mine += __popc(s_flags[w]);
    mine = warp_sum(mine);
    int total;
    int base = warp_prefix(mine, scratch.wtot[1], total);
    const uint32_t lt_mask = (1u << lane) - 1u;
    for (int w = w0; w < w1; ++w) {
        const uint32_t bits = s_flags[w];
        if ((bits >> lane) & 1u) idx[base + __popc(bits & lt_mask)] = (w << 5) + lane;
        base += __popc(bits);
    }
    if (threadIdx.x == 0) *count = total;
    if (bitmap != nullptr)
        for (int w = w0 + lane; w < w1; w += 32) bitmap[w] = s_flags[w];
}

// miss = A \ P (ascending), hit = |A & P|.  One block; each warp owns a contiguous run of
// list positions so that the output keeps A's order.  An entry outside [0, K) is neither a
// hit nor a miss; the status word reports it.
__global__ void __launch_bounds__(kSelectThreads, 1)
diff_kernel(const int32_t* __restrict__ idxA, const int32_t* __restrict__ cntA,
            const uint32_t* __restrict__ bitmapP, int K, int32_t* __restrict__ miss,
            int32_t* __restrict__ miss_count, int32_t* __restrict__ hit_count, int32_t* __restrict__ status) {
    __shared__ int scan[2][33];
    int n = *cntA;
    if (n < 0 || n > K) {
        if (threadIdx.x == 0) report_status(status, AFX_ERR_CAPACITY);
        n = max(0, min(n, K));
    }
    const int lane = lane_id();
    const uint32_t lt_mask = (1u << lane) - 1u;
    const int nchunks = (n + 31) >> 5;
    const int nw = blockDim.x >> 5;
    const int per = (nchunks + nw - 1) / nw;
    const int c0 = min(nchunks, warp_id() * per), c1 = min(nchunks, c0 + per);
    int cm = 0, cbad = 0;
    for (int c = c0; c < c1; ++c) {
        const int p = (c << 5) + lane;
        bool m = false, bad = false;
        if (p < n) {
            const int j = idxA[p];
            bad = static_cast<unsigned>(j) >= static_cast<unsigned>(K);
            m = !bad && ((bitmapP[j >> 5] >> (j & 31)) & 1u) == 0u;
        }
        cm += __popc(__ballot_sync(0xFFFFFFFFu, m));
        cbad += __popc(__ballot_sync(0xFFFFFFFFu, bad));
    }
    int total, total_bad;
    int base = warp_prefix(cm, scan[0], total);
    warp_prefix(cbad, scan[1], total_bad);
    for (int c = c0; c < c1; ++c) {
        const int p = (c << 5) + lane;
        bool m = false;
        int j = 0;
        if (p < n) {
            j = idxA[p];
            m = static_cast<unsigned>(j) < static_cast<unsigned>(K) && ((bitmapP[j >> 5] >> (j & 31)) & 1u) == 0u;
        }
        const uint32_t b = __ballot_sync(0xFFFFFFFFu, m);
        if (m) miss[base + __popc(b & lt_mask)] = j;
        base += __popc(b);
    }
    if (threadIdx.x == 0) {
        *miss_count = total;
        *hit_count = n - total - total_bad;
        if (total_bad > 0) report_status(status, AFX_ERR_INVALID_ARG);
    }
}

}  // namespace afx

extern "C" afx_status afx_select_active(const void* x, int dtype, int K, int T, int mode, int k,
                                        float tau, int32_t* idx, int32_t* count, uint32_t* bitmap,
                                        void* stream) {
    using namespace afx;
    if (x == nullptr || idx == nullptr || count == nullptr) return AFX_ERR_INVALID_ARG;
    if (K <= 0 || K > (1 << 20) || T < 1 || T > AFX_MAX_T) return AFX_ERR_INVALID_ARG;
    if (dtype != AFX_F16 && dtype != AFX_BF16) return AFX_ERR_UNSUPPORTED;
    if (mode != AFX_MODE_TOPK && mode != AFX_MODE_THRESHOLD) return AFX_ERR_UNSUPPORTED;
    if (mode == AFX_MODE_TOPK && (k < 0 || k > K)) return AFX_ERR_INVALID_ARG;
    if (mode == AFX_MODE_THRESHOLD && tau != tau) return AFX_ERR_INVALID_ARG;
    if ((reinterpret_cast<uintptr_t>(x) & 1u) || (reinterpret_cast<uintptr_t>(idx) & 3u) ||
        (reinterpret_cast<uintptr_t>(count) & 3u) || (reinterpret_cast<uintptr_t>(bitmap) & 3u))
        return AFX_ERR_ALIGNMENT;
    const size_t smem = select_dyn_smem(K);
    auto kern = dtype == AFX_F16 ? select_kernel<AFX_F16> : select_kernel<AFX_BF16>;
    if (!ensure_dyn_smem(reinterpret_cast<const void*>(kern), smem)) {
        cudaGetLastError();
        return AFX_ERR_CUDA;
    }
    kern<<<1, kSelectThreads, smem, static_cast<cudaStream_t>(stream)>>>(
        static_cast<const uint16_t*>(x), K, T, mode, k, tau, idx, count, bitmap);
    return launch_status();
}

extern "C" afx_status afx_diff_active(const int32_t* idxA, const int32_t* cntA,
                                      const uint32_t* bitmapP, int K, int32_t* miss,
                                      int32_t* miss_count, int32_t* hit_count, int32_t* dev_status,
                                      void* stream) {
    using namespace afx;
    if (idxA == nullptr || cntA == nullptr || bitmapP == nullptr || miss == nullptr ||
        miss_count == nullptr || hit_count == nullptr)
        return AFX_ERR_INVALID_ARG;
    if (K <= 0 || K > (1 << 20)) return AFX_ERR_INVALID_ARG;
    if ((reinterpret_cast<uintptr_t>(idxA) & 3u) || (reinterpret_cast<uintptr_t>(cntA) & 3u) ||
        (reinterpret_cast<uintptr_t>(bitmapP) & 3u) || (reinterpret_cast<uintptr_t>(miss) & 3u) ||
        (reinterpret_cast<uintptr_t>(miss_count) & 3u) || (reinterpret_cast<uintptr_t>(hit_count) & 3u) ||
        (reinterpret_cast<uintptr_t>(dev_status) & 3u))
        return AFX_ERR_ALIGNMENT;
    diff_kernel<<<1, kSelectThreads, 0, static_cast<cudaStream_t>(stream)>>>(
        idxA, cntA, bitmapP, K, miss, miss_count, hit_count, dev_status);
    return launch_status();
}
