// Arguments and launcher of the 4-bit sparse GEMV kernel (afx_q4.cu), shared with the layer
// step over 4-bit weights (afx_layer.cu).
#pragma once

#include <cuda_runtime.h>
#include <stdint.h>

#include <cooperative_groups.h>

#include "afx.h"
#include "afx_common.cuh"

namespace afx {

constexpr int kQ4Threads = 512;
constexpr int kQ4Warps = kQ4Threads / 32;
constexpr int kQ4Unroll = 8;   // 8-byte loads in flight per lane
constexpr int kQ4Cap = 1024;   // staged list entries per pass of the list kernel
constexpr int kQ4Opl = 16;     // outputs per lane and channel: half a block of 32

enum { Q4_STORE = 0, Q4_ACCUM = 1, Q4_SILU = 2 };

struct Q4Args {
    const unsigned char* Wq;
    int64_t ldq;  // row stride in bytes (multiple of 16)
    int K, N;
    const uint16_t* x;
    const int32_t* idx;
    const int32_t* count;
    // how a finished sum leaves: Q4_STORE y[i] = sum, Q4_ACCUM y[i] += sum; Q4_SILU: every block
    // of 32 outputs is 16 "gate" outputs (the low 4 bits of its 16 bytes) and 16 "up" outputs
    // (the high 4 bits), out_bits[16 b + m] = round(silu(gate_m) * up_m) in x's 16-bit type
    int ep;
    float* y;
    uint16_t* out_bits;
    int32_t* status;
};

// x_dtype AFX_F16 / AFX_BF16; arguments already validated.
afx_status launch_q4_list(int x_dtype, const Q4Args& a, cudaStream_t st);


// ---- device side: streaming loop and reduction shared by the list kernel and the fused operator ----

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

// Streams the staged channels [0, staged): s_off[p] = row offset in 16-byte units, s_x[p] = the
// channel's input value.  A lane owns 16 outputs of a channel: bytes 8h .. 8h+7 of a block's 16
// code bytes (h = half & 1), i.e. outputs 8h .. 8h+7 (low 4 bits) and 16+8h .. 16+8h+7 (high 4
// bits) of block half >> 1.  LPC lanes per channel piece: the tile is LPC * 16 outputs wide.
// acc: pairs (0,1) (2,3) (4,5) (6,7) of the low-nibble outputs, then of the high-nibble ones.
template <int LPC>
__device__ __forceinline__ void q4_stream(const unsigned char* Wq, int N, int half, const uint32_t* s_off,
                                          const float* s_x, int staged, f32x2 (&acc)[8]) {
    constexpr int SUB = 32 / LPC;        // channels per warp-wide load
    constexpr int EG = kQ4Warps * SUB;   // channel groups of the block
    const int lane = threadIdx.x & 31;
    const int eg = (threadIdx.x >> 5) * SUB + lane / LPC;
    const uint2* codes = reinterpret_cast<const uint2*>(Wq) + half;                           // + row offset * 2
    const uint16_t* scales = reinterpret_cast<const uint16_t*>(Wq + (N >> 1)) + (half >> 1);  // + row offset * 8
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

// Meeting of the sums of one tile -- lane groups of a warp, warps of the block, blocks of the
// cluster, in that fixed order -- and the epilogue `ep` (Q4_*).  s_red: (kQ4Warps + 1) * LPC * 16
// floats of shared memory, free on entry (a block barrier comes first).  Every thread of every
// block of the cluster calls it; no cluster barrier arrival may be pending.
template <int XDT, int LPC>
__device__ __forceinline__ void q4_finish(const f32x2 (&acc)[8], float* s_red, int tile, int N, int ep, float* y,
                                          uint16_t* out_bits) {
    namespace cg = cooperative_groups;
    constexpr int PW = LPC * kQ4Opl;
    cg::cluster_group cluster = cg::this_cluster();
    const int S = static_cast<int>(cluster.num_blocks());
    const int rank = static_cast<int>(cluster.block_rank());
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
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
    if (ep == Q4_SILU) {
        // pair r of the tile: gate = output 32 * (r / 16) + r % 16, up = 16 further on
        constexpr int HP = PW / 2;
        for (int r = rank + S * tid; r < HP; r += S * kQ4Threads) {
            const int og = (r >> 4) * 32 + (r & 15);
            const int m = tile * HP + r;
            if (2 * m < N) {
                float g = 0.0f, u = 0.0f;
                for (int q = 0; q < S; ++q) {
                    const float* pq = cluster.map_shared_rank(part, q);
                    g += pq[og];
                    u += pq[og + 16];
                }
                out_bits[m] = float_to_bits<XDT>(g / (1.0f + expf(-g)) * u);
            }
        }
    } else {
        for (int o = rank + S * tid; o < PW; o += S * kQ4Threads) {
            const int out = tile * PW + o;
            if (out < N) {
                float s = 0.0f;
                for (int q = 0; q < S; ++q) s += cluster.map_shared_rank(part, q)[o];
                y[out] = ep == Q4_ACCUM ? y[out] + s : s;
            }
        }
    }
    cluster.sync();  // peers may still be reading this block's sums
}

}  // namespace afx
