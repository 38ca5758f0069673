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

constexpr int kQ4Threads = 512;
constexpr int kQ4Warps = kQ4Threads / 32;
constexpr int kQ4Unroll = 8;   // 8-byte loads in flight per lane
constexpr int kQ4Cap = 1024;   // staged list entries per pass
constexpr int kQ4Opl = 16;     // outputs per lane and channel: half a block of 32

__device__ __forceinline__ uint2 ld_stream_8B(const void* p) {
    uint2 v;
    asm volatile("ld.global.nc.L1::no_allocate.v2.u32 {%0,%1}, [%2];" : "=r"(v.x), "=r"(v.y) : "l"(p));
    return v;
}
__device__ __forceinline__ f32x2 add_f32x2(f32x2 a, f32x2 b) {
    f32x2 r;
    asm("add.rn.f32x2 %0, %1, %2;" : "=l"(r) : "l"(a), "l"(b));
    return r;
}

// (code - 8) for the four codes in the low nibbles of v's bytes, as two fp32 pairs: a byte
// permute drops each code into the mantissa of 2^23 (0x4B0000qq = 2^23 + code), one two-wide
// add takes 2^23 + 8 away again.
__device__ __forceinline__ void nibbles_to_pairs(uint32_t v, f32x2& p01, f32x2& p23) {
    const uint32_t magic = 0x4B000000u;
    const f32x2 bias = pack_f32x2(-8388616.0f, -8388616.0f);
    f32x2 a, b;
    asm("mov.b64 %0, {%1, %2};" : "=l"(a) : "r"(__byte_perm(v, magic, 0x7540)), "r"(__byte_perm(v, magic, 0x7541)));
    asm("mov.b64 %0, {%1, %2};" : "=l"(b) : "r"(__byte_perm(v, magic, 0x7542)), "r"(__byte_perm(v, magic, 0x7543)));
    p01 = add_f32x2(a, bias);
    p23 = add_f32x2(b, bias);
}

// A lane owns 16 outputs of a channel: bytes 8h .. 8h+7 of a block's 16 code bytes (h = 0, 1),
// i.e. outputs 8h .. 8h+7 (low nibbles) and 16+8h .. 16+8h+7 (high nibbles) of the block.
// LPC lanes per channel piece: tile = LPC * 16 outputs.  Two blocks of 512 threads per SM.
template <int XDT, int LPC>
__global__ void __launch_bounds__(kQ4Threads, 2) sparse_gemv_q4_kernel(Q4Args a) {
    constexpr int SUB = 32 / LPC;        // channels per warp-wide load
    constexpr int EG = kQ4Warps * SUB;   // channel groups of the block
    constexpr int PW = LPC * kQ4Opl;     // outputs of the tile
    extern __shared__ __align__(16) unsigned char q4_dyn[];
    uint32_t* s_off = reinterpret_cast<uint32_t*>(q4_dyn);          // [kQ4Cap] row offset in 16-byte units
    float* s_x = reinterpret_cast<float*>(s_off + kQ4Cap);          // [kQ4Cap]
    float* s_red = s_x + kQ4Cap;                                    // [kQ4Warps][PW] then part[PW]
    __shared__ int first_ok;
    cg::cluster_group cluster = cg::this_cluster();
    const int S = static_cast<int>(cluster.num_blocks());
    const int rank = static_cast<int>(cluster.block_rank());
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
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
    const uint2* codes = reinterpret_cast<const uint2*>(a.Wq) + half;                               // + row offset * 2
    const uint16_t* scales = reinterpret_cast<const uint16_t*>(a.Wq + (a.N >> 1)) + (half >> 1);    // + row offset * 8
    const int eg = warp * SUB + lane / LPC;

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
        if (lane_ok) {
            for (int p = eg; p < staged; p += EG * kQ4Unroll) {
                uint2 raw[kQ4Unroll];
                uint16_t sc[kQ4Unroll];
#pragma unroll
                for (int u = 0; u < kQ4Unroll; ++u) {
                    const int pp = p + u * EG;
                    if (pp < staged) {
                        const uint32_t off = s_off[pp];
                        raw[u] = ld_stream_8B(codes + static_cast<size_t>(off) * 2);
                        sc[u] = __ldg(scales + static_cast<size_t>(off) * 8);
                    }
                }
#pragma unroll
                for (int u = 0; u < kQ4Unroll; ++u) {
                    const int pp = p + u * EG;
                    if (pp < staged) {
                        const float s = s_x[pp] * __half2float(__ushort_as_half(sc[u]));
                        const f32x2 s2 = pack_f32x2(s, s);
                        const uint32_t w[2] = {raw[u].x, raw[u].y};
#pragma unroll
                        for (int q = 0; q < 2; ++q) {  // word q: this lane's outputs 4q..4q+3 (low nibbles), 8+4q.. (high)
                            f32x2 a01, a23;
                            nibbles_to_pairs(w[q] & 0x0F0F0F0Fu, a01, a23);
                            fma_f32x2(acc[2 * q], a01, s2);
                            fma_f32x2(acc[2 * q + 1], a23, s2);
                            nibbles_to_pairs((w[q] >> 4) & 0x0F0F0F0Fu, a01, a23);
                            fma_f32x2(acc[4 + 2 * q], a01, s2);
                            fma_f32x2(acc[4 + 2 * q + 1], a23, s2);
                        }
                    }
                }
            }
        }
    }
    // ---- lane groups of a warp, warps of the block, blocks of the cluster: fixed order ----
    float v[kQ4Opl];
#pragma unroll
    for (int i = 0; i < 8; ++i) unpack_f32x2(acc[i], v[2 * i], v[2 * i + 1]);
#pragma unroll
    for (int o = LPC; o < 32; o <<= 1)
#pragma unroll
        for (int i = 0; i < kQ4Opl; ++i) v[i] += __shfl_xor_sync(0xFFFFFFFFu, v[i], o);
    __syncthreads();
    // position of this lane's 16 values inside the tile: block (lane / 2), bytes 8h..: outputs
    // 32 * blk + 8h + i (i < 8) and 32 * blk + 16 + 8h + i
    if (lane < LPC) {
        const int base = warp * PW + (lane >> 1) * 32 + (lane & 1) * 8;
        float4* lo4 = reinterpret_cast<float4*>(s_red + base);
        float4* hi4 = reinterpret_cast<float4*>(s_red + base + 16);
        lo4[0] = make_float4(v[0], v[1], v[2], v[3]);
        lo4[1] = make_float4(v[4], v[5], v[6], v[7]);
        hi4[0] = make_float4(v[8], v[9], v[10], v[11]);
        hi4[1] = make_float4(v[12], v[13], v[14], v[15]);
    }
    __syncthreads();
    float* part = s_red + kQ4Warps * PW;  // this block's sums, read by the cluster
    for (int o = tid; o < PW; o += kQ4Threads) {
        float s = 0.0f;
#pragma unroll
        for (int g = 0; g < kQ4Warps; ++g) s += s_red[g * PW + o];
        part[o] = s;
    }
    cluster.sync();
    if (a.ep == Q4_SILU) {
        // pair r of the tile: gate = output 32 * (r / 16) + r % 16, up = 16 further on
        constexpr int HP = PW / 2;
        for (int r = rank + S * tid; r < HP; r += S * kQ4Threads) {
            const int og = (r >> 4) * 32 + (r & 15);
            const int m = tile * HP + r;
            if (2 * m < a.N) {
                float g = 0.0f, u = 0.0f;
                for (int q = 0; q < S; ++q) {
                    const float* pq = cluster.map_shared_rank(part, q);
                    g += pq[og];
                    u += pq[og + 16];
                }
                a.out_bits[m] = float_to_bits<XDT>(g / (1.0f + expf(-g)) * u);
            }
        }
    } else {
        for (int o = rank + S * tid; o < PW; o += S * kQ4Threads) {
            const int out = tile * PW + o;
            if (out < a.N) {
                float s = 0.0f;
                for (int q = 0; q < S; ++q) s += cluster.map_shared_rank(part, q)[o];
                a.y[out] = a.ep == Q4_ACCUM ? a.y[out] + s : s;
            }
        }
    }
    cluster.sync();  // peers may still be reading this block's sums
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
