// Block-level active-channel selection: |x| top-k (two-pass radix select on the 15-bit
// magnitude key, ties to the lower channel id) or threshold, OR-ed over T tokens into a
// shared-memory bitmap, then an ordered compaction into an ascending index list.
//
// The routines are written for one thread block of whole warps (<= 32 warps) so that the
// stand-alone selection kernel and kernels that need the selection as a prologue can share
// them.  Every routine contains block-wide barriers: all threads of the block call it with
// the same arguments.
#pragma once

#include "afx_common.cuh"

namespace afx {

struct SelectScratch {
    int hist[256];
    int scan[33];
    int res[4];
};

// Words [w0, w1) of the bitmap owned by the calling warp (contiguous, so that a walk over
// warps in order visits channels in ascending order).
__device__ __forceinline__ void warp_word_range(int nwords, int& w0, int& w1) {
    const int nw = blockDim.x >> 5;
    const int per = (nwords + nw - 1) / nw;
    w0 = warp_id() * per;
    w1 = min(nwords, w0 + per);
    if (w0 > nwords) w0 = nwords;
}

// Warp 0 only.  hist has nbins (multiple of 32, <= 256) counters; walking bins from the
// highest down, finds the bin that holds the k-th element (k is 1-based and must not
// exceed the histogram's total).  res[0] = that bin, res[1] = number of elements in higher
// bins.
__device__ __forceinline__ void find_kth_bin(const int* hist, int nbins, int k, int* res) {
    const int per = nbins >> 5;
    const int l = lane_id();
    int local = 0;
    for (int q = 0; q < per; ++q) local += hist[nbins - 1 - (l * per + q)];
    int incl = local;
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) {
        int n = __shfl_up_sync(0xFFFFFFFFu, incl, o);
        if (l >= o) incl += n;
    }
    const int before = incl - local;
    if (before < k && k <= incl) {
        int run = before;
        for (int q = 0; q < per; ++q) {
            const int bin = nbins - 1 - (l * per + q);
            const int h = hist[bin];
            if (k <= run + h) {
                res[0] = bin;
                res[1] = run;
                break;
            }
            run += h;
        }
    }
}

// Fills flags[0..ceil(K/32)) (shared memory) with the union over tokens of the per-token
// active sets.  x is [T][K] in global memory.
template <int DT>
__device__ void block_select_flags(const uint16_t* __restrict__ x, int K, int T, int mode, int k,
                                   float tau, uint32_t* flags, SelectScratch* s) {
    const int nwords = (K + 31) >> 5;
    const int lane = lane_id();
    const uint32_t lt_mask = (1u << lane) - 1u;
    int w0, w1;
    warp_word_range(nwords, w0, w1);
    for (int w = w0 + lane; w < w1; w += 32) flags[w] = 0u;  // own range only
    __syncwarp();

    for (int t = 0; t < T; ++t) {
        const uint16_t* xt = x + static_cast<size_t>(t) * K;
        if (mode == AFX_MODE_THRESHOLD) {
            for (int w = w0; w < w1; ++w) {
                const int j = (w << 5) + lane;
                bool pred = false;
                if (j < K) pred = (tau < 0.0f) || (fabsf(bits_to_float<DT>(xt[j])) > tau);
                const uint32_t b = __ballot_sync(0xFFFFFFFFu, pred);
                if (lane == 0) flags[w] |= b;
            }
            continue;
        }
        // ---- top-k ----
        if (k <= 0) continue;
        if (k >= K) {
            for (int w = w0; w < w1; ++w) {
                const uint32_t b = __ballot_sync(0xFFFFFFFFu, (w << 5) + lane < K);
                if (lane == 0) flags[w] |= b;
            }
            continue;
        }
        // pass 1: histogram of the 8 high key bits
        __syncthreads();
        for (int i = threadIdx.x; i < 256; i += blockDim.x) s->hist[i] = 0;
        __syncthreads();
        for (int j = threadIdx.x; j < K; j += blockDim.x) atomicAdd(&s->hist[mag_key(xt[j]) >> 7], 1);
        __syncthreads();
        if (warp_id() == 0) find_kth_bin(s->hist, 256, k, s->res);
        __syncthreads();
        const uint32_t hi = static_cast<uint32_t>(s->res[0]);
        const int k2 = k - s->res[1];  // rank of the k-th element inside its high-bits bin
        // pass 2: histogram of the 7 low key bits inside that bin
        for (int i = threadIdx.x; i < 128; i += blockDim.x) s->hist[i] = 0;
        __syncthreads();
        for (int j = threadIdx.x; j < K; j += blockDim.x) {
            const uint32_t key = mag_key(xt[j]);
            if ((key >> 7) == hi) atomicAdd(&s->hist[key & 127u], 1);
        }
        __syncthreads();
        if (warp_id() == 0) find_kth_bin(s->hist, 128, k2, s->res + 2);
        __syncthreads();
        const uint32_t thr = (hi << 7) | static_cast<uint32_t>(s->res[2]);  // the k-th largest key
        const int need_eq = k2 - s->res[3];  // how many channels with key == thr are kept
        const bool all_eq = (need_eq == s->hist[s->res[2]]);
        if (all_eq) {
            for (int w = w0; w < w1; ++w) {
                const int j = (w << 5) + lane;
                const bool pred = j < K && mag_key(xt[j]) >= thr;
                const uint32_t b = __ballot_sync(0xFFFFFFFFu, pred);
                if (lane == 0) flags[w] |= b;
            }
        } else {
            // ties at the boundary: keep the need_eq lowest channel ids among key == thr
            int ce = 0;
            for (int w = w0; w < w1; ++w) {
                const int j = (w << 5) + lane;
                ce += __popc(__ballot_sync(0xFFFFFFFFu, j < K && mag_key(xt[j]) == thr));
            }
            int base = block_exclusive_over_warps(ce, s->scan);
            for (int w = w0; w < w1; ++w) {
                const int j = (w << 5) + lane;
                const uint32_t key = j < K ? mag_key(xt[j]) : 0u;
                const bool eq = j < K && key == thr;
                const uint32_t e = __ballot_sync(0xFFFFFFFFu, eq);
                const bool pred = j < K && (key > thr || (eq && base + __popc(e & lt_mask) < need_eq));
                const uint32_t b = __ballot_sync(0xFFFFFFFFu, pred);
                if (lane == 0) flags[w] |= b;
                base += __popc(e);
            }
        }
    }
    __syncthreads();
}

// Ordered compaction of a bitmap in shared memory: idx[0..total) = set bits ascending.
// idx may point to global or shared memory.  Returns the total (same in every thread).
__device__ __forceinline__ int block_compact_flags(const uint32_t* flags, int K, int32_t* idx,
                                                   SelectScratch* s) {
    const int nwords = (K + 31) >> 5;
    const int lane = lane_id();
    const uint32_t lt_mask = (1u << lane) - 1u;
    int w0, w1;
    warp_word_range(nwords, w0, w1);
    int c = 0;
    for (int w = w0 + lane; w < w1; w += 32) c += __popc(flags[w]);
    c = warp_sum(c);
    int base = block_exclusive_over_warps(c, s->scan);
    const int total = s->scan[32];
    for (int w = w0; w < w1; ++w) {
        const uint32_t bits = flags[w];
        if ((bits >> lane) & 1u) idx[base + __popc(bits & lt_mask)] = (w << 5) + lane;
        base += __popc(bits);
    }
    return total;
}

}  // namespace afx
