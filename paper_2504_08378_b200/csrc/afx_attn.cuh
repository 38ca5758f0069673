// Dense single-query attention over an fp16 KV cache for one decoding step (support op of
// the decoder layer; the paper keeps attention dense and so does this kernel).
//
// grid = (S, kv_heads, T), cluster = (S,1,1): the S blocks of a cluster split the L = pos+1
// cached positions of one (token, kv head) and meet their (max, sum, weighted V) partials
// through distributed shared memory.  The block owning the last position first rotates and
// stores the current token's k and v into the cache.  head_dim is fixed at 128.
#pragma once

#include <cooperative_groups.h>

#include "afx_common.cuh"

namespace afx {

namespace cg = cooperative_groups;

constexpr int kAttnThreads = 256;
constexpr int kAttnWarps = kAttnThreads / 32;
constexpr int kHeadDim = 128;
constexpr int kAttnKeyBlock = 256;
constexpr int kAttnMaxRep = 8;  // query heads per kv head
constexpr int kAttnUnroll = 4;  // cache rows in flight per half warp

struct AttnArgs {
    const float* qkv;  // [T][n_qkv] fp32: q heads | k heads | v heads
    int n_qkv, q_heads, kv_heads, T;
    uint16_t* k_cache;  // [T][max_seq][kv_heads][128] fp16 bits
    uint16_t* v_cache;
    int max_seq, pos;
    const float* rope_cos;  // [max_seq][64]
    const float* rope_sin;
    uint16_t* out;  // [T][q_heads*128] dtype bits
};

struct AttnSmem {
    float q[kAttnMaxRep][kHeadDim];
    float score[kAttnMaxRep][kAttnKeyBlock];
    __align__(16) float red[2 * kAttnWarps][kHeadDim];
    float m_new[kAttnMaxRep];
    float part_m[kAttnMaxRep];
    float part_l[kAttnMaxRep];
    float part_acc[kAttnMaxRep][kHeadDim];
};

__device__ __forceinline__ void unpack8_f16(const uint4& raw, float (&w)[8]) {
    const uint32_t r[4] = {raw.x, raw.y, raw.z, raw.w};
#pragma unroll
    for (int i = 0; i < 4; ++i) {
        const float2 f = __half22float2(*reinterpret_cast<const __half2*>(&r[i]));
        w[2 * i] = f.x;
        w[2 * i + 1] = f.y;
    }
}

template <int DT>
__device__ __forceinline__ void attention_block(const AttnArgs& a, AttnSmem* sm) {
    cg::cluster_group cluster = cg::this_cluster();
    const int S = static_cast<int>(cluster.num_blocks());
    const int rank = static_cast<int>(cluster.block_rank());
    const int hk = blockIdx.y, t = blockIdx.z;
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const int half = lane >> 4, l16 = lane & 15;
    const int rep = a.q_heads / a.kv_heads;
    const int L = a.pos + 1;
    const int l_lo = static_cast<int>(static_cast<int64_t>(rank) * L / S);
    const int l_hi = static_cast<int>(static_cast<int64_t>(rank + 1) * L / S);
    const float scale = rsqrtf(static_cast<float>(kHeadDim));
    const uint32_t half_mask = 0xFFFFu << (16 * half);  // the two halves of a warp work on different keys

    asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
    asm volatile("griddepcontrol.wait;" ::: "memory");

    const float* row = a.qkv + static_cast<size_t>(t) * a.n_qkv;
    const float* cs = a.rope_cos + static_cast<size_t>(a.pos) * (kHeadDim / 2);
    const float* sn = a.rope_sin + static_cast<size_t>(a.pos) * (kHeadDim / 2);
    uint16_t* kc = a.k_cache + static_cast<size_t>(t) * a.max_seq * a.kv_heads * kHeadDim;
    uint16_t* vc = a.v_cache + static_cast<size_t>(t) * a.max_seq * a.kv_heads * kHeadDim;
    const size_t row_stride = static_cast<size_t>(a.kv_heads) * kHeadDim;

    // rotated queries of this kv head's group
    for (int e = tid; e < rep * (kHeadDim / 2); e += kAttnThreads) {
        const int r = e / (kHeadDim / 2), i = e - r * (kHeadDim / 2);
        const float* qh = row + static_cast<size_t>(hk * rep + r) * kHeadDim;
        const float x0 = qh[2 * i], x1 = qh[2 * i + 1];
        sm->q[r][2 * i] = x0 * cs[i] - x1 * sn[i];
        sm->q[r][2 * i + 1] = x0 * sn[i] + x1 * cs[i];
    }
    // the block that owns the newest position appends the current k, v (fp16) first
    if (l_hi == L && l_lo < l_hi) {
        const float* kh = row + static_cast<size_t>(a.q_heads + hk) * kHeadDim;
        const float* vh = row + static_cast<size_t>(a.q_heads + a.kv_heads + hk) * kHeadDim;
        uint16_t* kdst = kc + static_cast<size_t>(a.pos) * row_stride + static_cast<size_t>(hk) * kHeadDim;
        uint16_t* vdst = vc + static_cast<size_t>(a.pos) * row_stride + static_cast<size_t>(hk) * kHeadDim;
        if (tid < kHeadDim / 2) {
            const float x0 = kh[2 * tid], x1 = kh[2 * tid + 1];
            kdst[2 * tid] = __half_as_ushort(__float2half_rn(x0 * cs[tid] - x1 * sn[tid]));
            kdst[2 * tid + 1] = __half_as_ushort(__float2half_rn(x0 * sn[tid] + x1 * cs[tid]));
        } else if (tid < kHeadDim / 2 + kHeadDim) {
            const int d = tid - kHeadDim / 2;
            vdst[d] = __half_as_ushort(__float2half_rn(vh[d]));
        }
    }
    __syncthreads();

    float m_run[kAttnMaxRep], l_run[kAttnMaxRep], acc[kAttnMaxRep][8];
#pragma unroll
    for (int r = 0; r < kAttnMaxRep; ++r) {
        m_run[r] = -INFINITY;
        l_run[r] = 0.0f;
#pragma unroll
        for (int j = 0; j < 8; ++j) acc[r][j] = 0.0f;
    }

    for (int b0 = l_lo; b0 < l_hi; b0 += kAttnKeyBlock) {
        const int nb = min(kAttnKeyBlock, l_hi - b0);
        // pass 1: scores of the block's keys (half a warp per key, kAttnUnroll keys in flight)
        for (int i0 = 2 * warp + half; i0 < nb; i0 += 2 * kAttnWarps * kAttnUnroll) {
            uint4 raw[kAttnUnroll];
#pragma unroll
            for (int u = 0; u < kAttnUnroll; ++u) {
                const int i = i0 + u * 2 * kAttnWarps;
                if (i < nb)
                    raw[u] = *reinterpret_cast<const uint4*>(kc + static_cast<size_t>(b0 + i) * row_stride +
                                                             static_cast<size_t>(hk) * kHeadDim + l16 * 8);
            }
#pragma unroll
            for (int u = 0; u < kAttnUnroll; ++u) {
                const int i = i0 + u * 2 * kAttnWarps;
                if (i < nb) {
                    float kv[8];
                    unpack8_f16(raw[u], kv);
#pragma unroll
                    for (int r = 0; r < kAttnMaxRep; ++r) {
                        if (r < rep) {
                            float d = 0.0f;
#pragma unroll
                            for (int j = 0; j < 8; ++j) d = fmaf(sm->q[r][l16 * 8 + j], kv[j], d);
                            d += __shfl_xor_sync(half_mask, d, 8);
                            d += __shfl_xor_sync(half_mask, d, 4);
                            d += __shfl_xor_sync(half_mask, d, 2);
                            d += __shfl_xor_sync(half_mask, d, 1);
                            if (l16 == 0) sm->score[r][i] = d * scale;
                        }
                    }
                }
            }
        }
        __syncthreads();
        // new running maximum per query head (warp r handles head r)
        if (warp < rep) {
            float mx = -INFINITY;
            for (int i = lane; i < nb; i += 32) mx = fmaxf(mx, sm->score[warp][i]);
#pragma unroll
            for (int o = 16; o > 0; o >>= 1) mx = fmaxf(mx, __shfl_xor_sync(0xFFFFFFFFu, mx, o));
            if (lane == 0) sm->m_new[warp] = mx;
        }
        __syncthreads();
        // pass 2: weights and weighted values
#pragma unroll
        for (int r = 0; r < kAttnMaxRep; ++r) {
            if (r < rep) {
                const float mn = fmaxf(m_run[r], sm->m_new[r]);
                const float f = expf(m_run[r] - mn);  // exp(-inf) = 0 on the first block
                l_run[r] *= f;
#pragma unroll
                for (int j = 0; j < 8; ++j) acc[r][j] *= f;
                m_run[r] = mn;
            }
        }
        for (int i0 = 2 * warp + half; i0 < nb; i0 += 2 * kAttnWarps * kAttnUnroll) {
            uint4 raw[kAttnUnroll];
#pragma unroll
            for (int u = 0; u < kAttnUnroll; ++u) {
                const int i = i0 + u * 2 * kAttnWarps;
                if (i < nb)
                    raw[u] = *reinterpret_cast<const uint4*>(vc + static_cast<size_t>(b0 + i) * row_stride +
                                                             static_cast<size_t>(hk) * kHeadDim + l16 * 8);
            }
#pragma unroll
            for (int u = 0; u < kAttnUnroll; ++u) {
                const int i = i0 + u * 2 * kAttnWarps;
                if (i < nb) {
                    float vv[8];
                    unpack8_f16(raw[u], vv);
#pragma unroll
                    for (int r = 0; r < kAttnMaxRep; ++r) {
                        if (r < rep) {
                            const float p = expf(sm->score[r][i] - m_run[r]);
                            l_run[r] += p;
#pragma unroll
                            for (int j = 0; j < 8; ++j) acc[r][j] = fmaf(p, vv[j], acc[r][j]);
                        }
                    }
                }
            }
        }
        __syncthreads();
    }

    // meet the 16 key groups of the block (fixed order), one query head at a time
#pragma unroll
    for (int r = 0; r < kAttnMaxRep; ++r) {
        if (r < rep) {
            float4* dst = reinterpret_cast<float4*>(&sm->red[2 * warp + half][l16 * 8]);
            dst[0] = make_float4(acc[r][0], acc[r][1], acc[r][2], acc[r][3]);
            dst[1] = make_float4(acc[r][4], acc[r][5], acc[r][6], acc[r][7]);
            if (l16 == 0) sm->score[0][2 * warp + half] = l_run[r];  // score[] is free now
            __syncthreads();
            if (tid < kHeadDim) {
                float s = 0.0f;
#pragma unroll
                for (int g = 0; g < 2 * kAttnWarps; ++g) s += sm->red[g][tid];
                sm->part_acc[r][tid] = s;
            } else if (tid == kHeadDim) {
                float s = 0.0f;
#pragma unroll
                for (int g = 0; g < 2 * kAttnWarps; ++g) s += sm->score[0][g];
                sm->part_l[r] = s;
                sm->part_m[r] = m_run[r];  // identical in every thread of the block
            }
            __syncthreads();
        }
    }
    cluster.sync();
    for (int e = rank + S * tid; e < rep * kHeadDim; e += S * kAttnThreads) {
        const int r = e / kHeadDim, d = e - r * kHeadDim;
        float M = -INFINITY;
        for (int q = 0; q < S; ++q) M = fmaxf(M, cluster.map_shared_rank(&sm->part_m[0], q)[r]);
        float num = 0.0f, den = 0.0f;
        for (int q = 0; q < S; ++q) {
            const float w = expf(cluster.map_shared_rank(&sm->part_m[0], q)[r] - M);
            num = fmaf(w, cluster.map_shared_rank(&sm->part_acc[0][0], q)[r * kHeadDim + d], num);
            den = fmaf(w, cluster.map_shared_rank(&sm->part_l[0], q)[r], den);
        }
        a.out[static_cast<size_t>(t) * a.q_heads * kHeadDim + static_cast<size_t>(hk * rep + r) * kHeadDim + d] =
            float_to_bits<DT>(num / den);
    }
    cluster.sync();
}

}  // namespace afx
