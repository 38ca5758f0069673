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
// A column is staged as its offset from the start of the weights in 16-byte units
// (row * ldw / 8: 32 bits cover operators of up to 64 GB), so that a load address is one
// multiply-add away.
template <int TMAX, int CAP>
struct GemvSmem {
    uint32_t col[CAP];
    float xv[TMAX][CAP];
    __align__(16) float red[kGemvWarps][256];  // per-warp sums of one token
};

// Where the blocks of a cluster deliver their partial sums: block q owns every S-th output
// (or gate/up pair) of the tile and receives one value per (source block, token, owned
// output).  Written by remote blocks while this block may still be in any phase of its own
// work, so it must not share storage with anything else.
constexpr int kRecvPerToken = 272;  // >= PW + 2 * kMaxCluster - 2
template <int TMAX>
struct GemvRecv {
    float v[TMAX * kRecvPerToken];
};

// Split cluster barrier.  Every block arrives once when it starts and waits just before its
// first store into a peer's shared memory: by then every block of the cluster is running.
__device__ __forceinline__ void cluster_arrive() {
    asm volatile("barrier.cluster.arrive.release.aligned;" ::: "memory");
}
__device__ __forceinline__ void cluster_wait() {
    asm volatile("barrier.cluster.wait.acquire.aligned;" ::: "memory");
}

// How a finished sum leaves the kernel.
enum { EP_STORE = 0, EP_ACCUM = 1, EP_SILU = 2 };

struct EpilogueArgs {
    float* y;            // EP_STORE / EP_ACCUM: [T][N] fp32
    uint16_t* out_bits;  // EP_SILU: [T][N/2] 16-bit floats
    int N;               // outputs of the operator (columns of Wt)
    const float* scale;  // EP_STORE / EP_ACCUM: DEVICE factor applied to the finished sum (an
                         // expert's routing weight), or NULL for 1
};

// Streams the staged channels [0, staged) of one tile: acc[t][q] += xv[t][p] * W[row(p)][out0+q].
// wbase16 points at this lane's 8 outputs of row 0; sm->col[p] is row(p)'s offset in 16-byte
// units.  Products and sums are two-wide fused multiply-adds (bitwise the scalar fma.rn
// results).  SPLIT: full batches of U loads per lane run without per-load guards and a guarded
// batch finishes (fewer instructions; the extra loop costs registers, which the fused operator
// kernels with their selection state do not have to spare).
template <int DT, int TMAX, int PW, int CAP, bool SPLIT>
__device__ __forceinline__ void gemv_stream(const uint4* __restrict__ wbase16, int T,
                                            const GemvSmem<TMAX, CAP>* sm, int staged,
                                            float (&acc)[TMAX][8]) {
    constexpr int LPC = PW / 8;             // lanes per channel piece
    constexpr int SUB = 32 / LPC;           // channel pieces per warp-wide load
    constexpr int EG = kGemvWarps * SUB;    // channel groups in the block
    constexpr int U = kGemvUnroll;
    const int lane = threadIdx.x & 31;
    const int eg = (threadIdx.x >> 5) * SUB + lane / LPC;
    f32x2 a2[TMAX][4];
#pragma unroll
    for (int t = 0; t < TMAX; ++t)
#pragma unroll
        for (int i = 0; i < 4; ++i) a2[t][i] = pack_f32x2(acc[t][2 * i], acc[t][2 * i + 1]);
    auto consume = [&](const uint4& raw, int pp) {
        f32x2 w[4];
        unpack8_pairs<DT>(raw, w);
#pragma unroll
        for (int t = 0; t < TMAX; ++t) {
            if (t < T) {
                const float xv = sm->xv[t][pp];
                const f32x2 x2 = pack_f32x2(xv, xv);
#pragma unroll
                for (int i = 0; i < 4; ++i) fma_f32x2(a2[t][i], w[i], x2);
            }
        }
    };
    // one batch: U loads per lane in flight, then their products
    auto batch = [&](int p, bool guarded) {
        uint4 raw[U];
#pragma unroll
        for (int u = 0; u < U; ++u)
            if (!guarded || p + u * EG < staged) raw[u] = ld_stream_16B(wbase16 + sm->col[p + u * EG]);
#pragma unroll
        for (int u = 0; u < U; ++u)
            if (!guarded || p + u * EG < staged) consume(raw[u], p + u * EG);
    };
    if (SPLIT) {
        int p = eg;
        for (; p + (U - 1) * EG < staged; p += EG * U) batch(p, false);
        if (p < staged) batch(p, true);
    } else {
        for (int p = eg; p < staged; p += EG * U) batch(p, true);
    }
#pragma unroll
    for (int t = 0; t < TMAX; ++t)
#pragma unroll
        for (int i = 0; i < 4; ++i) unpack_f32x2(a2[t][i], acc[t][2 * i], acc[t][2 * i + 1]);
}

// Block-level then cluster-level meeting of the sums of one tile, then the epilogue:
//   EP_STORE  y[t][out]  = sum            EP_ACCUM  y[t][out] += sum
//   EP_SILU   columns come in groups of 16 = 8 "gate" then 8 "up" outputs;
//             out_bits[t][m] = round(silu(gate_m) * up_m) for the N/2 pairs m.
// Block q of the cluster finishes the outputs (pairs) o with o % S == q: every block pushes
// its partial sums into the owners' GemvRecv through distributed shared memory, one cluster
// barrier later each owner adds the S contributions in rank order.  Every thread of every
// block of the cluster must call this, after one cluster_arrive() earlier in the kernel whose
// wait is still pending (pending_wait) or has been taken by the caller since.
template <int DT, int TMAX, int PW, int CAP, int EP>
__device__ __forceinline__ void gemv_finish_tile(float (&acc)[TMAX][8], int T, int tile,
                                                 GemvSmem<TMAX, CAP>* sm, GemvRecv<TMAX>* recv,
                                                 const EpilogueArgs& ep, bool pending_wait = true) {
    constexpr int LPC = PW / 8;
    constexpr int HP = PW / 2;  // gate/up pairs per tile
    const int lane = threadIdx.x & 31;
    const int warp = threadIdx.x >> 5;
    cg::cluster_group cluster = cg::this_cluster();
    const int S = static_cast<int>(cluster.num_blocks());
    const int rank = static_cast<int>(cluster.block_rank());
    const int W = EP == EP_SILU ? 2 * ((HP + S - 1) / S) : (PW + S - 1) / S;  // values per (source, token)
    // where this thread's output goes: owner block and slot inside the owner's row
    int owner = 0, slot = 0;
    if (threadIdx.x < PW) {
        const int o = threadIdx.x;
        if (EP == EP_SILU) {
            const int r = (o >> 4) * 8 + (o & 7);  // pair index; bit 3 of o says gate (0) / up (1)
            owner = r % S;
            slot = (r / S) * 2 + ((o >> 3) & 1);
        } else {
            owner = o % S;
            slot = o / S;
        }
    }
    float* dst = cluster.map_shared_rank(&recv->v[0], owner);
    // EP_ACCUM: the value this thread will add to (first element it finishes) is asked for now,
    // so that its latency passes behind the reduction and the cluster barrier
    float y_old = 0.0f;
    if (EP == EP_ACCUM && threadIdx.x < T * W) {
        const int t = threadIdx.x / W, sl = threadIdx.x - t * W;
        const int o = sl * S + rank;
        const int out = tile * PW + o;
        if (o < PW && out < ep.N) y_old = ep.y[static_cast<size_t>(t) * ep.N + out];
    }
    if (pending_wait) cluster_wait();  // pairs with the cluster_arrive() at kernel start: all peers are running
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
                float4* d4 = reinterpret_cast<float4*>(&sm->red[warp][lane * 8]);
                d4[0] = make_float4(acc[t][0], acc[t][1], acc[t][2], acc[t][3]);
                d4[1] = make_float4(acc[t][4], acc[t][5], acc[t][6], acc[t][7]);
            }
            __syncthreads();
            if (threadIdx.x < PW) {
                float s = 0.0f;
#pragma unroll
                for (int g = 0; g < kGemvWarps; ++g) s += sm->red[g][threadIdx.x];
                dst[(rank * T + t) * W + slot] = s;
            }
        }
    }
    const float out_scale = (EP != EP_SILU && ep.scale != nullptr) ? *ep.scale : 1.0f;
    cluster.sync();  // every contribution has landed
    const float* mine = &recv->v[0];
    if (EP == EP_SILU) {
        const int WP = W / 2;
        for (int e = threadIdx.x; e < T * WP; e += kGemvThreads) {
            const int t = e / WP, ps = e - t * WP;
            const int r = ps * S + rank;
            const int m = tile * HP + r;
            if (r < HP && 2 * m < ep.N) {
                float g = 0.0f, u = 0.0f;
                for (int q = 0; q < S; ++q) {
                    g += mine[(q * T + t) * W + 2 * ps];
                    u += mine[(q * T + t) * W + 2 * ps + 1];
                }
                const float v = g / (1.0f + expf(-g)) * u;
                ep.out_bits[static_cast<size_t>(t) * (ep.N / 2) + m] = float_to_bits<DT>(v);
            }
        }
    } else {
        for (int e = threadIdx.x; e < T * W; e += kGemvThreads) {
            const int t = e / W, sl = e - t * W;
            const int o = sl * S + rank;
            const int out = tile * PW + o;
            if (o < PW && out < ep.N) {
                float s = 0.0f;
                for (int q = 0; q < S; ++q) s += mine[(q * T + t) * W + sl];
                s *= out_scale;
                float* p = ep.y + static_cast<size_t>(t) * ep.N + out;
                *p = (EP == EP_ACCUM) ? (e < kGemvThreads ? y_old : *p) + s : s;
            }
        }
    }
}

constexpr uint32_t kSkippedEntry = 0xFFFFFFFFu;  // staged column of a list entry that takes no part

struct GemvListArgs {
    const uint16_t* Wt;
    int64_t ldw;
    int K, N, T;
    const uint16_t* x;
    const int32_t* idx;
    const int32_t* count;
    const int32_t* slot;
    int accumulate;   // 0: y = sum, 1: y += sum
    int silu;         // 1: gate|up columns, out_bits = round(silu(gate) * up) instead of y
    EpilogueArgs ep;
    int32_t* status;  // device status word or NULL
};

// afx_sparse_gemv's launcher (afx_gemv.cu), also used by the layer step over host-resident weights.
afx_status launch_list_gemv(int dtype, const GemvListArgs& a, cudaStream_t st);

// grid = (S, tiles), cluster = (S, 1, 1).
template <int DT, int TMAX, int PW, int CAP>
__device__ __forceinline__ void gemv_list_block(const GemvListArgs& a, GemvSmem<TMAX, CAP>* sm,
                                                GemvRecv<TMAX>* recv) {
    constexpr int LPC = PW / 8;
    const int tid = threadIdx.x;
    const int lane = tid & 31;
    const int S = gridDim.x, s = blockIdx.x, tile = blockIdx.y;
    const int T = a.T;
    cluster_arrive();
    // Programmatic dependent launch: global memory is touched only once the previous grid is
    // complete, and the next grid in the stream may be scheduled (as SM resources free up)
    // only after that -- so whatever a grid reads before its own wait was written at least
    // two grids earlier and is complete.
    asm volatile("griddepcontrol.wait;" ::: "memory");
    asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
    int cnt = *a.count;
    if (cnt < 0 || cnt > a.K) {
        if (tid == 0 && s == 0 && tile == 0) report_status(a.status, AFX_ERR_CAPACITY);
        cnt = max(0, min(cnt, a.K));
    }
    const int c_lo = static_cast<int>(static_cast<int64_t>(s) * cnt / S);
    const int c_hi = static_cast<int>(static_cast<int64_t>(s + 1) * cnt / S);
    const int out0 = tile * PW + (lane % LPC) * 8;
    const bool lane_ok = out0 < a.N;
    const uint64_t ld16 = static_cast<uint64_t>(a.ldw >> 3);  // row stride in 16-byte units
    const uint4* wbase16 = reinterpret_cast<const uint4*>(a.Wt + out0);

    float acc[TMAX][8];
#pragma unroll
    for (int t = 0; t < TMAX; ++t)
#pragma unroll
        for (int q = 0; q < 8; ++q) acc[t][q] = 0.0f;

    __shared__ int first_ok;
    for (int c0 = c_lo; c0 < c_hi; c0 += CAP) {
        int staged = min(CAP, c_hi - c0);
        __syncthreads();
        bool skipped = false;
        for (int i = tid; i < staged; i += kGemvThreads) {
            // An entry outside [0, K), or one whose cache slot is negative (a channel that found
            // no row), takes no part: x = 0, and the status word says so.
            const int j = a.idx[c0 + i];
            const int col = a.slot != nullptr ? a.slot[c0 + i] : j;
            const bool in_range = static_cast<unsigned>(j) < static_cast<unsigned>(a.K);
            const uint64_t off = static_cast<uint64_t>(col < 0 ? 0 : col) * ld16;
            const bool ok = in_range && col >= 0 && off + static_cast<uint64_t>(a.N >> 3) <= 0xFFFFFFFFull;
            if (!ok && tile == 0) report_status(a.status, in_range ? AFX_ERR_CAPACITY : AFX_ERR_INVALID_ARG);
            skipped |= !ok;
            sm->col[i] = ok ? static_cast<uint32_t>(off) : kSkippedEntry;
#pragma unroll
            for (int t = 0; t < TMAX; ++t)
                if (t < T) sm->xv[t][i] = ok ? bits_to_float<DT>(a.x[static_cast<size_t>(t) * a.K + j]) : 0.0f;
        }
        if (__syncthreads_or(skipped)) {
            // Rare.  A skipped entry still costs a load in the streaming loop; whatever it reads
            // is multiplied by 0, so it must read weights (finite), not a row nobody filled:
            // send it to the column of the first entry that does take part.
            if (tid == 0) first_ok = staged;
            __syncthreads();
            for (int i = tid; i < staged; i += kGemvThreads)
                if (sm->col[i] != kSkippedEntry) atomicMin(&first_ok, i);
            __syncthreads();
            const int f = first_ok;
            if (f < staged) {
                const uint32_t safe = sm->col[f];
                __syncthreads();
                for (int i = tid; i < staged; i += kGemvThreads)
                    if (sm->col[i] == kSkippedEntry) sm->col[i] = safe;
            } else {
                staged = 0;  // nothing in this part of the list takes part
            }
            __syncthreads();
        }
        if (lane_ok) gemv_stream<DT, TMAX, PW, CAP, true>(wbase16, T, sm, staged, acc);
    }
    if (a.silu)
        gemv_finish_tile<DT, TMAX, PW, CAP, EP_SILU>(acc, T, tile, sm, recv, a.ep);
    else if (a.accumulate)
        gemv_finish_tile<DT, TMAX, PW, CAP, EP_ACCUM>(acc, T, tile, sm, recv, a.ep);
    else
        gemv_finish_tile<DT, TMAX, PW, CAP, EP_STORE>(acc, T, tile, sm, recv, a.ep);
}

}  // namespace afx
