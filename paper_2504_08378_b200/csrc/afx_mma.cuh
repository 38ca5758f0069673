// Sparse GEMV for a few tokens at once (2 <= T <= 8) on the tensor cores.
//
// With T tokens every weight is multiplied T times.  On the fp32 pipe that is 4 T two-wide
// multiply-adds per 16-byte load and the loop is bound by instruction issue (at T = 8 by the fp32
// pipe itself); as a matrix product  D[outputs][tokens] = W^T[outputs][channels] . X[channels][tokens]
// the same work is one `mma` per 16 outputs x 16 channels x 8 tokens and the loop is bound by
// HBM again.  The contraction runs over the ACTIVE channels only: their rows are gathered from
// global memory into shared memory (16-byte asynchronous copies, several stages in flight), read
// back transposed as A fragments (`ldmatrix.trans`: a row of shared memory is one channel, the
// fragment wants one output per row), and meet the tokens' 16-bit inputs as B fragments.
// Products of two 16-bit floats are exact; the sums are fp32 inside the tensor core, in a fixed
// order: the same inputs give the same bits.
//
// A cluster of S blocks owns a tile of 256 outputs (16 warps x 16 outputs) and splits the active
// list; partial sums meet through distributed shared memory in rank order.
#pragma once

#include <cooperative_groups.h>

#include "afx_gemv.cuh"

namespace afx {

constexpr int kMtTokens = 8;                      // token rows of the B operand (rows >= T hold zeros)
constexpr int kMtTile = 256;                      // outputs per cluster
constexpr int kMtRowBytes = kMtTile * 2 + 16;     // a staged channel row (+16 bytes: ldmatrix rows fall into different banks)
constexpr int kMtPartStride = kMtTile + 4;        // floats per token row of the partial sums

// CAPM = staged list entries per pass (a multiple of ROWS): every pass fills and drains
// the pipeline once, so a block that is alone on its SM takes a large one.
// STAGES = pipeline stages (STAGES - 1 of them in flight while one is multiplied).
// ROWS = channels per stage (a multiple of 16).
template <int CAPM, int STAGES, int ROWS = 32>
struct MtSmem {
    static constexpr int kCap = CAPM;
    static constexpr int kStages = STAGES;
    static constexpr int kRows = ROWS;
    static constexpr int kStageBytes = ROWS * kMtRowBytes;
    static_assert(ROWS % 16 == 0 && CAPM % ROWS == 0 && kMtTokens * kMtPartStride * 4 <= ROWS * kMtRowBytes,
                  "stage shape (the partial sums reuse the first stage buffer)");
    uint32_t col[CAPM];                                // row offset of a staged channel in 16-byte units
    __align__(16) uint16_t xb[kMtTokens][CAPM + 8];    // the tokens' inputs at the staged channels (+16 bytes per row: no bank conflicts)
    __align__(16) unsigned char w[STAGES][ROWS * kMtRowBytes];
};

__device__ __forceinline__ uint32_t mt_smem_u32(const void* p) {
    return static_cast<uint32_t>(__cvta_generic_to_shared(p));
}
// 16 bytes global -> shared (dst = shared-window address); src_bytes = 0 writes zeros and reads nothing
__device__ __forceinline__ void mt_copy16(uint32_t dst, const void* src, uint32_t src_bytes) {
    asm volatile("cp.async.cg.shared.global [%0], [%1], 16, %2;" ::"r"(dst), "l"(src), "r"(src_bytes) : "memory");
}
__device__ __forceinline__ void mt_commit() { asm volatile("cp.async.commit_group;" ::: "memory"); }
template <int N>
__device__ __forceinline__ void mt_wait() {
    asm volatile("cp.async.wait_group %0;" ::"n"(N) : "memory");
}

template <int DT>
__device__ __forceinline__ void mt_mma(float (&c)[4], const uint32_t (&a)[4], uint32_t b0, uint32_t b1) {
    if (DT == AFX_F16)
        asm volatile("mma.sync.aligned.m16n8k16.row.col.f32.f16.f16.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%0,%1,%2,%3};"
                     : "+f"(c[0]), "+f"(c[1]), "+f"(c[2]), "+f"(c[3])
                     : "r"(a[0]), "r"(a[1]), "r"(a[2]), "r"(a[3]), "r"(b0), "r"(b1));
    else
        asm volatile("mma.sync.aligned.m16n8k16.row.col.f32.bf16.bf16.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%0,%1,%2,%3};"
                     : "+f"(c[0]), "+f"(c[1]), "+f"(c[2]), "+f"(c[3])
                     : "r"(a[0]), "r"(a[1]), "r"(a[2]), "r"(a[3]), "r"(b0), "r"(b1));
}

// One pass over the staged channels [0, staged) (sm->col, sm->xb filled, zero x behind `staged`
// up to the end of the last stage, a block barrier since): kStages - 1 stages of kRows
// channels in flight while one is multiplied.  wtile16 = the weights at this tile's first output;
// n_chunks = valid 16-byte pieces per row of the tile (pieces beyond the operator's last output
// and rows at or beyond `staged` are filled with zeros).  Every thread of the block calls it; on
// return all copies have landed.  Everything that does not depend on the stage is computed once:
// a thread copies the same 16-byte piece of two rows of every stage, a lane reads the same
// fragment positions of every stage.
template <int DT, class SMT>
__device__ __forceinline__ void mt_stream_pass(const uint4* wtile16, SMT* sm, int staged, int n_chunks, float (&c)[4]) {
    constexpr int kSt = SMT::kStages;
    constexpr int kMtStageRows = SMT::kRows;
    constexpr int kMtStageBytes = SMT::kStageBytes;
    constexpr int kChunks = kMtTile / 8;                       // 16-byte pieces per row
    constexpr int kSweep = kGemvThreads / kChunks;             // rows the block copies at once
    static_assert(kChunks == 32 && kMtStageRows % kSweep == 0, "copy pattern");
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const int gid = lane >> 2, tig = lane & 3;
    const int r0 = tid / kChunks, ch = tid % kChunks;
    const bool ch_ok = ch < n_chunks;
    const uint4* src_base = wtile16 + ch;
    const uint32_t w_base = mt_smem_u32(sm->w[0]);
    const uint32_t dst0 = w_base + r0 * kMtRowBytes + ch * 16;
    // lane l gives the address of row l % 8 of matrix l / 8: matrices (channels 0-7 | 8-15) x (outputs 0-7 | 8-15)
    const uint32_t a0 = w_base + ((lane >> 4) * 8 + (lane & 7)) * kMtRowBytes + (warp * 16 + ((lane >> 3) & 1) * 8) * 2;
    const uint32_t x0 = mt_smem_u32(&sm->xb[gid][2 * tig]);
    const int n_st = (staged + kMtStageRows - 1) / kMtStageRows;

    auto request = [&](int q, int buf) {
        if (q < n_st) {
#pragma unroll
            for (int i = 0; i < kMtStageRows / kSweep; ++i) {
                const int p = q * kMtStageRows + r0 + i * kSweep;
                const bool valid = ch_ok && p < staged;
                const uint4* src = valid ? src_base + sm->col[p] : wtile16;
                mt_copy16(dst0 + buf * kMtStageBytes + i * kSweep * kMtRowBytes, src, valid ? 16u : 0u);
            }
        }
        mt_commit();
    };
    auto multiply = [&](int q, int buf) {
#pragma unroll
        for (int k0 = 0; k0 < kMtStageRows; k0 += 16) {
            uint32_t a[4], b0, b1;
            asm volatile("ldmatrix.sync.aligned.m8n8.x4.trans.shared.b16 {%0,%1,%2,%3}, [%4];"
                         : "=r"(a[0]), "=r"(a[1]), "=r"(a[2]), "=r"(a[3])
                         : "r"(a0 + buf * kMtStageBytes + k0 * kMtRowBytes));
            const uint32_t xa = x0 + (q * kMtStageRows + k0) * 2;
            asm volatile("ld.shared.u32 %0, [%1];" : "=r"(b0) : "r"(xa));
            asm volatile("ld.shared.u32 %0, [%1];" : "=r"(b1) : "r"(xa + 16));
            mt_mma<DT>(c, a, b0, b1);
        }
    };
#pragma unroll
    for (int j = 0; j < kSt - 1; ++j) request(j, j);
    for (int q0 = 0; q0 < n_st; q0 += kSt) {
#pragma unroll
        for (int j = 0; j < kSt; ++j) {  // stage q0 + j lives in buffer j
            const int q = q0 + j;
            if (q < n_st) {
                mt_wait<kSt - 2>();  // stage q has landed (this thread's copies)
                __syncthreads();     // ... everybody's; and stage q - 1 has been multiplied by everybody
                request(q + kSt - 1, (j + kSt - 1) % kSt);
                multiply(q, j);
            }
        }
    }
    mt_wait<0>();
}

// Zeros behind the staged entries of the T token rows up to the end of the last stage, and the
// token rows that hold no token: whatever the multiply reads there must be 0 (no barrier).
template <class SMT>
__device__ __forceinline__ void mt_pad_inputs(SMT* sm, int T, int staged) {
    constexpr int kMtStageRows = SMT::kRows;
    const int padded = (staged + kMtStageRows - 1) / kMtStageRows * kMtStageRows;
    for (int i = staged + threadIdx.x; i < padded; i += kGemvThreads)
        for (int t = 0; t < T; ++t) sm->xb[t][i] = 0;
    for (int t = T; t < kMtTokens; ++t)
        for (int i = threadIdx.x; i < padded; i += kGemvThreads) sm->xb[t][i] = 0;
}

// The cluster's partial sums meet in rank order, then the epilogue (EP_STORE / EP_ACCUM /
// EP_SILU as in gemv_finish_tile).  Every thread of every block of the cluster calls it; no
// cluster barrier arrival may be pending.
// S blocks of the cluster, ranks base .. base + S - 1, worked on this tile; the caller is the
// rank-th of them (S < 0: the whole cluster).
template <int DT, class SMT>
__device__ __forceinline__ void mt_finish(const float (&c)[4], SMT* sm, int T, int tile, int N, int ep_kind,
                                          const EpilogueArgs& ep, int S = -1, int rank = 0, int base = 0) {
    namespace cg = cooperative_groups;
    cg::cluster_group cluster = cg::this_cluster();
    if (S < 0) {
        S = static_cast<int>(cluster.num_blocks());
        rank = static_cast<int>(cluster.block_rank());
    }
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    __syncthreads();  // the last stage has been multiplied by everybody
    float* part = reinterpret_cast<float*>(sm->w[0]);  // [8 tokens][kMtPartStride]
    {
        const int gid = lane >> 2, tig = lane & 3, o = warp * 16 + gid;
        part[(2 * tig) * kMtPartStride + o] = c[0];
        part[(2 * tig + 1) * kMtPartStride + o] = c[1];
        part[(2 * tig) * kMtPartStride + o + 8] = c[2];
        part[(2 * tig + 1) * kMtPartStride + o + 8] = c[3];
    }
    cluster.sync();
    if (ep_kind == EP_SILU) {
        // columns in groups of 16 = 8 gate then 8 up outputs: pair r of the tile
        constexpr int HP = kMtTile / 2;
        for (int e = rank + S * tid; e < T * HP; e += S * kGemvThreads) {
            const int t = e / HP, r = e - t * HP;
            const int og = (r >> 3) * 16 + (r & 7);
            const int m = tile * HP + r;
            if (2 * m < N) {
                float g = 0.0f, u = 0.0f;
                for (int q = 0; q < S; ++q) {
                    const float* pq = cluster.map_shared_rank(part, base + q) + t * kMtPartStride;
                    g += pq[og];
                    u += pq[og + 8];
                }
                ep.out_bits[static_cast<size_t>(t) * (N / 2) + m] = float_to_bits<DT>(g / (1.0f + expf(-g)) * u);
            }
        }
    } else {
        const float out_scale = ep.scale != nullptr ? *ep.scale : 1.0f;
        for (int e = rank + S * tid; e < T * kMtTile; e += S * kGemvThreads) {
            const int t = e / kMtTile, o = e - t * kMtTile;
            const int out = tile * kMtTile + o;
            if (out < N) {
                float s = 0.0f;
                for (int q = 0; q < S; ++q) s += cluster.map_shared_rank(part, base + q)[t * kMtPartStride + o];
                s *= out_scale;
                float* p = ep.y + static_cast<size_t>(t) * N + out;
                *p = ep_kind == EP_ACCUM ? *p + s : s;
            }
        }
    }
    cluster.sync();  // peers may still be reading this block's sums
}

// grid = (S, tiles of 256 outputs), cluster = (S, 1, 1), 512 threads.
template <int DT, class SMT>
__device__ __forceinline__ void mt_list_block(const GemvListArgs& a, SMT* sm) {
    constexpr int kMtCap = SMT::kCap;
    namespace cg = cooperative_groups;
    cg::cluster_group cluster = cg::this_cluster();
    const int S = static_cast<int>(cluster.num_blocks());
    const int rank = static_cast<int>(cluster.block_rank());
    const int tid = threadIdx.x;
    const int tile = blockIdx.y, T = a.T;
    asm volatile("griddepcontrol.wait;" ::: "memory");
    asm volatile("griddepcontrol.launch_dependents;" ::: "memory");  // only after the wait (ordering rule of the library)
    int cnt = *a.count;
    if (cnt < 0 || cnt > a.K) {
        if (tid == 0 && rank == 0 && tile == 0) report_status(a.status, AFX_ERR_CAPACITY);
        cnt = max(0, min(cnt, a.K));
    }
    const int c_lo = static_cast<int>(static_cast<int64_t>(rank) * cnt / S);
    const int c_hi = static_cast<int>(static_cast<int64_t>(rank + 1) * cnt / S);
    const uint64_t ld16 = static_cast<uint64_t>(a.ldw >> 3);
    const uint4* wtile16 = reinterpret_cast<const uint4*>(a.Wt + static_cast<size_t>(tile) * kMtTile);
    const int n_chunks = min(kMtTile, a.N - tile * kMtTile) >> 3;

    float c[4] = {0.0f, 0.0f, 0.0f, 0.0f};
    __shared__ int first_ok;

    for (int c0 = c_lo; c0 < c_hi; c0 += kMtCap) {
        int staged = min(kMtCap, c_hi - c0);
        __syncthreads();  // the previous pass has been multiplied
        bool skipped = false;
        for (int i = tid; i < staged; i += kGemvThreads) {
            // as in the fp32 kernel: an entry outside [0, K) or with a negative cache slot takes no part
            const int j = a.idx[c0 + i];
            const int col = a.slot != nullptr ? a.slot[c0 + i] : j;
            const bool in_range = static_cast<unsigned>(j) < static_cast<unsigned>(a.K);
            const uint64_t off = static_cast<uint64_t>(col < 0 ? 0 : col) * ld16;
            const bool ok = in_range && col >= 0 && off + static_cast<uint64_t>(a.N >> 3) <= 0xFFFFFFFFull;
            if (!ok && tile == 0) report_status(a.status, in_range ? AFX_ERR_CAPACITY : AFX_ERR_INVALID_ARG);
            skipped |= !ok;
            sm->col[i] = ok ? static_cast<uint32_t>(off) : kSkippedEntry;
            for (int t = 0; t < T; ++t) sm->xb[t][i] = ok ? a.x[static_cast<size_t>(t) * a.K + j] : uint16_t(0);
        }
        mt_pad_inputs(sm, T, staged);
        if (__syncthreads_or(skipped)) {  // rare: a skipped entry reads the row of one that takes part (x = 0)
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
                staged = 0;
            }
            __syncthreads();
        }
        mt_stream_pass<DT>(wtile16, sm, staged, n_chunks, c);
    }
    mt_finish<DT>(c, sm, T, tile, a.N, a.silu ? EP_SILU : (a.accumulate ? EP_ACCUM : EP_STORE), a.ep);
}

}  // namespace afx
