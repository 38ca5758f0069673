// Sparse GEMV over an active-channel list: y[t][i] = sum_c x[t][idx[c]] * Wt[col(c)][i].
//
// Work decomposition.  The outputs are cut into column tiles of PW (256, 128 or 64) values;
// a thread-block CLUSTER of S blocks owns one tile and its S blocks take S equal contiguous
// parts of the active list, so every block of the grid streams the same number of bytes and
// the grid is a single wave.  Inside a block each lane owns 8 consecutive outputs (one
// 128-bit load per channel), PW/8 lanes cover one channel's piece of the tile, and the
// 16 warps (times 32/(PW/8) lane groups) take alternate channels with fp32 accumulators in
// registers.  Sums meet in three fixed-order steps: lane groups by warp shuffle, warps in
// shared memory, the cluster's blocks through distributed shared memory.  No global
// scratch, no atomics: the same inputs give the same bits.
#pragma once

#include <cooperative_groups.h>

#include "afx_common.cuh"

namespace afx {

namespace cg = cooperative_groups;

constexpr int kGemvWarps = 16;
constexpr int kGemvThreads = 32 * kGemvWarps;
constexpr int kGemvUnroll = 8;
constexpr int kMaxCluster = 8;

// Shared memory of one block.  CAP = channels whose (column, x) pairs are staged at once.
template <int TMAX, int CAP>
struct GemvSmem {
    int col[CAP];
    float xv[TMAX][CAP];
    __align__(16) float red[kGemvWarps][256];  // per-warp sums of one token
    __align__(16) float part[TMAX][256];       // this block's sums, read by the cluster
};

// How a finished sum leaves the kernel.
enum { EP_STORE = 0, EP_ACCUM = 1, EP_SILU = 2 };

struct EpilogueArgs {
    float* y;            // EP_STORE / EP_ACCUM: [T][N] fp32
    uint16_t* out_bits;  // EP_SILU: [T][N/2] 16-bit floats
    int N;               // outputs of the operator (columns of Wt)
};

// Streams the staged channels [0, staged) of one tile: acc[t][q] += xv[t][p] * W[col[p]][out0+q].
template <int DT, int TMAX, int PW, int CAP>
__device__ __forceinline__ void gemv_stream(const uint16_t* __restrict__ wbase, int64_t ldw, int T,
                                            const GemvSmem<TMAX, CAP>* sm, int staged,
                                            float (&acc)[TMAX][8]) {
    constexpr int LPC = PW / 8;             // lanes per channel piece
    constexpr int SUB = 32 / LPC;           // channel pieces per warp-wide load
    constexpr int EG = kGemvWarps * SUB;    // channel groups in the block
    constexpr int U = kGemvUnroll;
    const int lane = threadIdx.x & 31;
    const int eg = (threadIdx.x >> 5) * SUB + lane / LPC;
    for (int p = eg; p < staged; p += EG * U) {
        uint4 raw[U];
#pragma unroll
        for (int u = 0; u < U; ++u) {
            const int pp = p + u * EG;
            if (pp < staged) raw[u] = ld_stream_16B(wbase + static_cast<int64_t>(sm->col[pp]) * ldw);
        }
#pragma unroll
        for (int u = 0; u < U; ++u) {
            const int pp = p + u * EG;
            if (pp < staged) {
                float w[8];
                unpack8<DT>(raw[u], w);
#pragma unroll
                for (int t = 0; t < TMAX; ++t) {
                    if (t < T) {
                        const float xv = sm->xv[t][pp];
#pragma unroll
                        for (int q = 0; q < 8; ++q) acc[t][q] = fmaf(xv, w[q], acc[t][q]);
                    }
                }
            }
        }
    }
}

// Block-level then cluster-level meeting of the sums of one tile, then the epilogue:
//   EP_STORE  y[t][out]  = sum            EP_ACCUM  y[t][out] += sum
//   EP_SILU   columns come in groups of 16 = 8 "gate" then 8 "up" outputs;
//             out_bits[t][m] = round(silu(gate_m) * up_m) for the N/2 pairs m.
// Each (token, output) is finished by exactly one thread of the cluster.  Every thread of
// every block of the cluster must call this (it holds cluster barriers).
template <int DT, int TMAX, int PW, int CAP, int EP>
__device__ __forceinline__ void gemv_finish_tile(float (&acc)[TMAX][8], int T, int tile,
                                                 GemvSmem<TMAX, CAP>* sm, const EpilogueArgs& ep) {
    constexpr int LPC = PW / 8;
    const int lane = threadIdx.x & 31;
    const int warp = threadIdx.x >> 5;
    cg::cluster_group cluster = cg::this_cluster();
    const int S = static_cast<int>(cluster.num_blocks());
    const int rank = static_cast<int>(cluster.block_rank());
#pragma unroll
    for (int t = 0; t < TMAX; ++t) {
        if (t < T) {
            // lane groups of a warp hold different channels of the same outputs
#pragma unroll
            for (int o = LPC; o < 32; o <<= 1)
#pragma unroll
                for (int q = 0; q < 8; ++q) acc[t][q] += __shfl_xor_sync(0xFFFFFFFFu, acc[t][q], o);
            __syncthreads();
            if (lane < LPC) {
                float4* dst = reinterpret_cast<float4*>(&sm->red[warp][lane * 8]);
                dst[0] = make_float4(acc[t][0], acc[t][1], acc[t][2], acc[t][3]);
                dst[1] = make_float4(acc[t][4], acc[t][5], acc[t][6], acc[t][7]);
            }
            __syncthreads();
            if (threadIdx.x < PW) {
                float s = 0.0f;
#pragma unroll
                for (int g = 0; g < kGemvWarps; ++g) s += sm->red[g][threadIdx.x];
                sm->part[t][threadIdx.x] = s;
            }
        }
    }
    cluster.sync();  // every block's part[][] is complete and visible
    const float* parts[kMaxCluster];
#pragma unroll
    for (int q = 0; q < kMaxCluster; ++q)
        parts[q] = q < S ? cluster.map_shared_rank(&sm->part[0][0], q) : nullptr;
    if (EP == EP_SILU) {
        constexpr int HP = PW / 2;  // pairs per tile
        const int total = T * HP;
        for (int e = rank + S * static_cast<int>(threadIdx.x); e < total; e += S * kGemvThreads) {
            const int t = e / HP, r = e - t * HP;
            const int og = (r >> 3) * 16 + (r & 7);
            const int m = tile * HP + r;
            if (2 * m < ep.N) {
                float g = 0.0f, u = 0.0f;
#pragma unroll
                for (int q = 0; q < kMaxCluster; ++q)
                    if (q < S) {
                        g += parts[q][t * 256 + og];
                        u += parts[q][t * 256 + og + 8];
                    }
                const float v = g / (1.0f + expf(-g)) * u;
                ep.out_bits[static_cast<size_t>(t) * (ep.N / 2) + m] = float_to_bits<DT>(v);
            }
        }
    } else {
        const int total = T * PW;
        for (int e = rank + S * static_cast<int>(threadIdx.x); e < total; e += S * kGemvThreads) {
            const int t = e / PW, o = e - t * PW;
            const int out = tile * PW + o;
            if (out < ep.N) {
                float s = 0.0f;
#pragma unroll
                for (int q = 0; q < kMaxCluster; ++q)
                    if (q < S) s += parts[q][t * 256 + o];
                float* p = ep.y + static_cast<size_t>(t) * ep.N + out;
                *p = (EP == EP_ACCUM) ? *p + s : s;
            }
        }
    }
    cluster.sync();  // nobody leaves while its shared memory may still be read
}

struct GemvListArgs {
    const uint16_t* Wt;
    int64_t ldw;
    int K, N, T;
    const uint16_t* x;
    const int32_t* idx;
    const int32_t* count;
    const int32_t* slot;
    int accumulate;
    EpilogueArgs ep;
};

// grid = (S, tiles), cluster = (S, 1, 1).
template <int DT, int TMAX, int PW, int CAP>
__device__ __forceinline__ void gemv_list_block(const GemvListArgs& a, GemvSmem<TMAX, CAP>* sm) {
    constexpr int LPC = PW / 8;
    const int tid = threadIdx.x;
    const int lane = tid & 31;
    const int S = gridDim.x, s = blockIdx.x, tile = blockIdx.y;
    const int T = a.T;
    // Programmatic dependent launch: let the next grid in the stream be scheduled as soon as
    // SM resources free up, and touch global memory only once the previous grid is complete.
    asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
    asm volatile("griddepcontrol.wait;" ::: "memory");
    int cnt = *a.count;
    cnt = max(0, min(cnt, a.K));
    const int c_lo = static_cast<int>(static_cast<int64_t>(s) * cnt / S);
    const int c_hi = static_cast<int>(static_cast<int64_t>(s + 1) * cnt / S);
    const int out0 = tile * PW + (lane % LPC) * 8;
    const bool lane_ok = out0 < a.N;

    float acc[TMAX][8];
#pragma unroll
    for (int t = 0; t < TMAX; ++t)
#pragma unroll
        for (int q = 0; q < 8; ++q) acc[t][q] = 0.0f;

    for (int c0 = c_lo; c0 < c_hi; c0 += CAP) {
        const int staged = min(CAP, c_hi - c0);
        __syncthreads();
        for (int i = tid; i < staged; i += kGemvThreads) {
            const int j = a.idx[c0 + i];
            sm->col[i] = a.slot != nullptr ? a.slot[c0 + i] : j;
#pragma unroll
            for (int t = 0; t < TMAX; ++t)
                if (t < T) sm->xv[t][i] = bits_to_float<DT>(a.x[static_cast<size_t>(t) * a.K + j]);
        }
        __syncthreads();
        if (lane_ok) gemv_stream<DT, TMAX, PW, CAP>(a.Wt + out0, a.ldw, T, sm, staged, acc);
    }
    if (a.accumulate)
        gemv_finish_tile<DT, TMAX, PW, CAP, EP_ACCUM>(acc, T, tile, sm, a.ep);
    else
        gemv_finish_tile<DT, TMAX, PW, CAP, EP_STORE>(acc, T, tile, sm, a.ep);
}

}  // namespace afx
