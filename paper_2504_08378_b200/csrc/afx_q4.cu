// afx_sparse_gemv_q4: sparse GEMV over 4-bit block-quantised, channel-contiguous weights
// (Sec. 6: the weights are stored transposed so that a channel's scaling factors are read with
// the channel; Sec. 7.1: every evaluated model is 4-bit).
//
// A channel's row is [N/2 bytes of 4-bit codes][N/32 fp16 scales]; a block of 32 outputs is 16
// bytes of codes and one scale: byte m = code of output m (low 4 bits) and of output 16 + m
// (high 4 bits); value = (code - 8) * scale.  One lane owns HALF a block of one channel per
// load: an 8-byte read of the codes plus the block's scale, x * scale once, then 16
// multiply-adds with the codes turned into fp32 by a byte permute into the mantissa of 2^23
// (0x4B0000qq = 2^23 + q) and a subtraction of 2^23 + 8 -- two-wide adds and fused
// multiply-adds.  The tile of a cluster is LPC half blocks (LPC * 16 outputs) wide; the S blocks
// of the cluster split the active list and meet through distributed shared memory in rank
// order; sums are fp32 in a fixed order.  3.5x fewer bytes per weight than the 16-bit kernels,
// but 5-6 executed instructions per weight: this kernel is bound by instruction issue, not by
// HBM (64 registers, two 512-thread blocks per SM).
#include <cooperative_groups.h>

#include "afx_launch.cuh"
#include "afx_q4.cuh"

namespace afx {

namespace cg = cooperative_groups;

// A lane owns 16 outputs of a channel: bytes 8h .. 8h+7 of a block's 16 code bytes (h = 0, 1),
// i.e. outputs 8h .. 8h+7 (low nibbles) and 16+8h .. 16+8h+7 (high nibbles) of the block.
// LPC lanes per channel piece: tile = LPC * 16 outputs.  Two blocks of 512 threads per SM.
template <int XDT, int LPC>
__global__ void __launch_bounds__(kQ4Threads, 2) sparse_gemv_q4_kernel(Q4Args a) {
    extern __shared__ __align__(16) unsigned char q4_dyn[];
    uint32_t* s_off = reinterpret_cast<uint32_t*>(q4_dyn);          // [kQ4Cap] row offset in 16-byte units
    float* s_x = reinterpret_cast<float*>(s_off + kQ4Cap);          // [kQ4Cap]
    float* s_red = s_x + kQ4Cap;                                    // [kQ4Warps][PW] then part[PW]
    __shared__ int first_ok;
    cg::cluster_group cluster = cg::this_cluster();
    const int S = static_cast<int>(cluster.num_blocks());
    const int rank = static_cast<int>(cluster.block_rank());
    const int tid = threadIdx.x, lane = tid & 31;
    const int tile = blockIdx.y;
    asm volatile("griddepcontrol.wait;" ::: "memory");
    asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
    int cnt = *a.count;
    if (cnt < 0 || cnt > a.K) {
        if (tid == 0 && rank == 0 && tile == 0) report_status(a.status, AFX_ERR_CAPACITY);
        cnt = max(0, min(cnt, a.K));
    }
    const int c_lo = static_cast<int>(static_cast<int64_t>(rank) * cnt / S);
    const int c_hi = static_cast<int>(static_cast<int64_t>(rank + 1) * cnt / S);
    const int half = tile * LPC + (lane % LPC);  // this lane's half block: block half >> 1, bytes 8 * (half & 1) ..
    const bool lane_ok = half * kQ4Opl < a.N;
    const uint64_t ld16 = static_cast<uint64_t>(a.ldq >> 4);

    f32x2 acc[8];  // pairs (0,1) (2,3) (4,5) (6,7) of the low nibbles, then of the high nibbles
#pragma unroll
    for (int i = 0; i < 8; ++i) acc[i] = pack_f32x2(0.0f, 0.0f);

    for (int c0 = c_lo; c0 < c_hi; c0 += kQ4Cap) {
        int staged = min(kQ4Cap, c_hi - c0);
        __syncthreads();
        bool skipped = false;
        for (int i = tid; i < staged; i += kQ4Threads) {
            const int j = a.idx[c0 + i];
            const uint64_t off = static_cast<uint64_t>(j < 0 ? 0 : j) * ld16;
            const bool ok = static_cast<unsigned>(j) < static_cast<unsigned>(a.K) && off + ld16 <= 0xFFFFFFFFull;
            if (!ok && tile == 0) report_status(a.status, AFX_ERR_INVALID_ARG);
            skipped |= !ok;
            s_off[i] = ok ? static_cast<uint32_t>(off) : 0xFFFFFFFFu;
            s_x[i] = ok ? bits_to_float<XDT>(a.x[j]) : 0.0f;
        }
        if (__syncthreads_or(skipped)) {  // rare: a skipped entry reads the row of one that takes part
            if (tid == 0) first_ok = staged;
            __syncthreads();
            for (int i = tid; i < staged; i += kQ4Threads)
                if (s_off[i] != 0xFFFFFFFFu) atomicMin(&first_ok, i);
            __syncthreads();
            const int f = first_ok;
            if (f < staged) {
                const uint32_t safe = s_off[f];
                __syncthreads();
                for (int i = tid; i < staged; i += kQ4Threads)
                    if (s_off[i] == 0xFFFFFFFFu) s_off[i] = safe;
            } else {
                staged = 0;
            }
            __syncthreads();
        }
        if (lane_ok) q4_stream<LPC>(a.Wq, a.N, half, s_off, s_x, staged, acc);
    }
    q4_finish<XDT, LPC>(acc, s_red, tile, a.N, a.ep, a.y, a.out_bits);
}

static size_t q4_dyn_smem(int lpc) {
    return static_cast<size_t>(kQ4Cap) * 8 + static_cast<size_t>(kQ4Warps + 1) * lpc * kQ4Opl * 4;
}

template <int XDT>
static afx_status launch_q4(const Q4Args& a, cudaStream_t st) {
    const void* kerns[3] = {reinterpret_cast<const void*>(sparse_gemv_q4_kernel<XDT, 32>),
                            reinterpret_cast<const void*>(sparse_gemv_q4_kernel<XDT, 16>),
                            reinterpret_cast<const void*>(sparse_gemv_q4_kernel<XDT, 8>)};
    const int lpcs[3] = {32, 16, 8};
    // the widest tile and largest cluster that keep every cluster resident at once, most blocks wins
    int best = 2, best_S = 1, best_blocks = -1;
    for (int i = 0; i < 3; ++i) {
        const int tiles = (a.N + lpcs[i] * kQ4Opl - 1) / (lpcs[i] * kQ4Opl);
        const size_t dyn = q4_dyn_smem(lpcs[i]);
        for (int S = kMaxCluster; S >= 1; --S) {
            const int margin = (tiles + 15) / 16 < 2 ? 2 : (tiles + 15) / 16;
            if (max_active_clusters(kerns[i], S, dyn, kQ4Threads) >= tiles + margin) {
                if (tiles * S > best_blocks) {
                    best_blocks = tiles * S;
                    best = i;
                    best_S = S;
                }
                break;
            }
        }
    }
    const int lpc = lpcs[best];
    const int tiles = (a.N + lpc * kQ4Opl - 1) / (lpc * kQ4Opl);
    if (tiles > 65535) return AFX_ERR_CAPACITY;
    const size_t dyn = q4_dyn_smem(lpc);
    switch (lpc) {
        case 32: return launch_clustered(sparse_gemv_q4_kernel<XDT, 32>, best_S, tiles, dyn, a, st, kQ4Threads);
        case 16: return launch_clustered(sparse_gemv_q4_kernel<XDT, 16>, best_S, tiles, dyn, a, st, kQ4Threads);
        default: return launch_clustered(sparse_gemv_q4_kernel<XDT, 8>, best_S, tiles, dyn, a, st, kQ4Threads);
    }
}

afx_status launch_q4_list(int x_dtype, const Q4Args& a, cudaStream_t st) {
    return x_dtype == AFX_F16 ? launch_q4<AFX_F16>(a, st) : launch_q4<AFX_BF16>(a, st);
}

}  // namespace afx

extern "C" size_t afx_q4_row_bytes(int N) {
    if (N < 32 || (N & 31) != 0) return 0;
    return (static_cast<size_t>(N) / 2 + static_cast<size_t>(N) / 16 + 15) / 16 * 16;
}

extern "C" afx_status afx_sparse_gemv_q4(const void* Wq, int K, int N, int64_t ldq_bytes, const void* x, int x_dtype,
                                         const int32_t* idx, const int32_t* count, float* y, int accumulate,
                                         int32_t* dev_status, void* stream) {
    using namespace afx;
    if (Wq == nullptr || x == nullptr || idx == nullptr || count == nullptr || y == nullptr) return AFX_ERR_INVALID_ARG;
    if (K <= 0 || N <= 0) return AFX_ERR_INVALID_ARG;
    if (x_dtype != AFX_F16 && x_dtype != AFX_BF16) return AFX_ERR_UNSUPPORTED;
    if ((N & 31) != 0 || (ldq_bytes & 15) != 0 || !aligned16(Wq) || (reinterpret_cast<uintptr_t>(y) & 3u) != 0 ||
        (reinterpret_cast<uintptr_t>(x) & 1u) != 0 || (reinterpret_cast<uintptr_t>(idx) & 3u) != 0 ||
        (reinterpret_cast<uintptr_t>(count) & 3u) != 0 || (reinterpret_cast<uintptr_t>(dev_status) & 3u) != 0)
        return AFX_ERR_ALIGNMENT;
    if (ldq_bytes < static_cast<int64_t>(afx_q4_row_bytes(N))) return AFX_ERR_INVALID_ARG;
    Q4Args a = {};
    a.Wq = static_cast<const unsigned char*>(Wq);
    a.ldq = ldq_bytes;
    a.K = K;
    a.N = N;
    a.x = static_cast<const uint16_t*>(x);
    a.idx = idx;
    a.count = count;
    a.y = y;
    a.ep = accumulate ? Q4_ACCUM : Q4_STORE;
    a.status = dev_status;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    return launch_q4_list(x_dtype, a, st);
}
