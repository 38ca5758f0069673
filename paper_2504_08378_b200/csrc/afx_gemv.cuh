// Sparse GEMV over an active-channel list: y[t][i] = sum_c x[t][idx[c]] * Wt[col(c)][i].
//
// Work decomposition.  The (active channel, output) plane is cut into column tiles of
// TW = WN*256 outputs; tile-major, the tiles' channel lists form one flat sequence of
// F = tiles * cnt "row pieces" (one piece = TW contiguous 16-bit weights of one channel).
// The G resident thread blocks split that sequence into G equal contiguous ranges, so every
// block streams the same number of bytes whatever cnt and N are, and the whole grid is one
// wave.  Inside a block, WC warp groups take alternate pieces, each lane owning 8
// consecutive outputs (one 128-bit load per piece) with fp32 accumulators in registers;
// the groups' sums meet in shared memory.  A tile covered by several blocks is finished by
// the last block to arrive (ticket counter, no waiting): it adds the blocks' partial sums in
// block order, so the result does not depend on timing.
#pragma once

#include "afx_common.cuh"

namespace afx {

constexpr int kPieceW = 256;       // outputs per warp-wide piece: 32 lanes x 8 weights

struct GemvArgs {
    const uint16_t* Wt;
    int64_t ldw;
    int K, N, T;
    const uint16_t* x;
    const int32_t* idx;
    const int32_t* count;
    const int32_t* slot;
    float* y;
    int accumulate;
    float* partials;  // [(G + tiles)][T][TW]
    int* counters;    // [tiles], zero between calls
};

// CAP = row pieces whose (column, x) pairs are staged in shared memory at once.
template <int CAP>
struct GemvShared {
    int col[CAP];
    int ticket;
};

// First and last block (inclusive) whose range meets tile `t`; ranges are
// [floor(b*F/G), floor((b+1)*F/G)).
__device__ __forceinline__ void tile_contributors(int64_t F, int64_t G, int64_t cnt, int t,
                                                  int& b_first, int& b_last) {
    const int64_t X = static_cast<int64_t>(t) * cnt, Y = X + cnt;
    b_first = static_cast<int>(((X + 1) * G + F - 1) / F - 1);
    b_last = static_cast<int>((Y * G + F - 1) / F - 1);
}

template <int DT, int TMAX, int WN, int WC, int U, int CAP>
__device__ __forceinline__ void gemv_block(const GemvArgs& a, GemvShared<CAP>* sh, float* s_x /*[TMAX][CAP]*/,
                                           float* s_red /*[WC][WN*256]*/) {
    constexpr int TW = WN * kPieceW;
    constexpr int NTHREADS = 32 * WN * WC;
    const int tid = threadIdx.x;
    const int lane = tid & 31;
    const int wn = (tid >> 5) % WN;   // which 256-wide part of the tile
    const int wc = (tid >> 5) / WN;   // which channel group
    const int T = a.T;

    int cnt = *a.count;
    cnt = max(0, min(cnt, a.K));
    const int tiles = (a.N + TW - 1) / TW;
    if (cnt == 0) {
        if (!a.accumulate) {
            const int64_t total = static_cast<int64_t>(T) * a.N;
            for (int64_t i = static_cast<int64_t>(blockIdx.x) * NTHREADS + tid; i < total;
                 i += static_cast<int64_t>(gridDim.x) * NTHREADS)
                a.y[i] = 0.0f;
        }
        return;
    }
    const int64_t F = static_cast<int64_t>(tiles) * cnt;
    const int64_t G = min64(gridDim.x, F);
    const int b = blockIdx.x;
    if (b >= G) return;
    const int64_t f0 = (b * F) / G, f1 = ((b + 1) * F) / G;

    float acc[TMAX][8];
#pragma unroll
    for (int t = 0; t < TMAX; ++t)
#pragma unroll
        for (int e = 0; e < 8; ++e) acc[t][e] = 0.0f;

    for (int64_t e0 = f0; e0 < f1; e0 += CAP) {
        const int64_t e1 = min64(f1, e0 + CAP);
        const int staged = static_cast<int>(e1 - e0);
        // ---- stage (column, x values) of the pieces [e0, e1) ----
        __syncthreads();
        for (int i = tid; i < staged; i += NTHREADS) {
            const int c = static_cast<int>((e0 + i) % cnt);
            const int j = a.idx[c];
            sh->col[i] = a.slot != nullptr ? a.slot[c] : j;
#pragma unroll
            for (int t = 0; t < TMAX; ++t)
                if (t < T) s_x[t * CAP + i] = bits_to_float<DT>(a.x[static_cast<size_t>(t) * a.K + j]);
        }
        __syncthreads();

        int64_t e = e0;
        while (e < e1) {
            const int tile = static_cast<int>(e / cnt);
            const int64_t tile_begin = static_cast<int64_t>(tile) * cnt;
            const int64_t tile_end = tile_begin + cnt;
            const int64_t s1 = min64(e1, tile_end);
            const int out0 = tile * TW + wn * kPieceW + lane * 8;
            const bool lane_ok = out0 < a.N;
            // ---- stream this block's pieces of the tile ----
            if (lane_ok) {
                const uint16_t* wbase = a.Wt + out0;
                const int lo = static_cast<int>(e - e0), hi = static_cast<int>(s1 - e0);
                for (int p = lo + wc; p < hi; p += WC * U) {
                    uint4 raw[U];
#pragma unroll
                    for (int u = 0; u < U; ++u) {
                        const int pp = p + u * WC;
                        if (pp < hi) raw[u] = ld_stream_16B(wbase + static_cast<int64_t>(sh->col[pp]) * a.ldw);
                    }
#pragma unroll
                    for (int u = 0; u < U; ++u) {
                        const int pp = p + u * WC;
                        if (pp < hi) {
                            float w[8];
                            unpack8<DT>(raw[u], w);
#pragma unroll
                            for (int t = 0; t < TMAX; ++t) {
                                if (t < T) {
                                    const float xv = s_x[t * CAP + pp];
#pragma unroll
                                    for (int q = 0; q < 8; ++q) acc[t][q] = fmaf(xv, w[q], acc[t][q]);
                                }
                            }
                        }
                    }
                }
            }
            const bool seg_done = (s1 == tile_end) || (s1 == f1);
            if (seg_done) {
                const int64_t seg_begin = max64(f0, tile_begin);
                const bool whole = (seg_begin == tile_begin) && (s1 == tile_end);
                int b_first = b, b_last = b;
                if (!whole) tile_contributors(F, G, cnt, tile, b_first, b_last);
                const int n_contrib = b_last - b_first + 1;
                float* my_partial = a.partials + static_cast<size_t>(b + tile) * T * TW;
                // ---- meet the WC groups' sums in shared memory, one token at a time ----
#pragma unroll
                for (int t = 0; t < TMAX; ++t) {
                    if (t < T) {
                        __syncthreads();
                        float4* dst = reinterpret_cast<float4*>(s_red + wc * TW + wn * kPieceW + lane * 8);
                        dst[0] = make_float4(acc[t][0], acc[t][1], acc[t][2], acc[t][3]);
                        dst[1] = make_float4(acc[t][4], acc[t][5], acc[t][6], acc[t][7]);
                        __syncthreads();
                        for (int o = tid; o < TW; o += NTHREADS) {
                            float s = 0.0f;
#pragma unroll
                            for (int g = 0; g < WC; ++g) s += s_red[g * TW + o];
                            const int out = tile * TW + o;
                            if (n_contrib == 1) {
                                if (out < a.N) {
                                    float* yp = a.y + static_cast<size_t>(t) * a.N + out;
                                    *yp = a.accumulate ? *yp + s : s;
                                }
                            } else {
                                my_partial[t * TW + o] = s;
                            }
                        }
                    }
#pragma unroll
                    for (int q = 0; q < 8; ++q) acc[t][q] = 0.0f;
                }
                if (n_contrib > 1) {
                    // ---- publish the partial; the last block to arrive finishes the tile ----
                    __threadfence();
                    __syncthreads();
                    if (tid == 0) sh->ticket = atomicAdd(&a.counters[tile], 1);
                    __syncthreads();
                    if (sh->ticket == n_contrib - 1) {
                        __threadfence();
                        const float* p0 = a.partials + static_cast<size_t>(b_first + tile) * T * TW;
                        for (int i = tid; i < T * TW; i += NTHREADS) {
                            const int t = i / TW, o = i - t * TW;
                            const int out = tile * TW + o;
                            if (out < a.N) {
                                float s = 0.0f;
                                for (int g = 0; g < n_contrib; ++g)
                                    s += __ldcg(p0 + static_cast<size_t>(g) * T * TW + i);
                                float* yp = a.y + static_cast<size_t>(t) * a.N + out;
                                *yp = a.accumulate ? *yp + s : s;
                            }
                        }
                        if (tid == 0) a.counters[tile] = 0;
                    }
                }
            }
            e = s1;
        }
    }
}

}  // namespace afx
