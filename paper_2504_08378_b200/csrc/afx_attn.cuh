// Dense single-query attention over an fp16 KV cache for one decoding step (support op of
// the decoder layer; the paper keeps attention dense and so does this kernel).
//
// grid = (S, kv_heads, T), cluster = (S,1,1): the S blocks of a cluster split the L = pos+1
// cached positions of one (token, kv head) and meet their (max, sum, weighted V) partials
// through distributed shared memory (softmax in base 2: exp(s) = 2^(s * log2 e)).  The block owning the last position first rotates and
// stores the current token's k and v into the cache.  head_dim is fixed at 128.
#pragma once

#include <cooperative_groups.h>

#include "afx_common.cuh"

namespace afx {

namespace cg = cooperative_groups;

constexpr int kAttnThreads = 256;
constexpr int kAttnWarps = kAttnThreads / 32;
constexpr int kAttnWorkers = 2 * kAttnWarps;  // half warps: each walks its own positions
constexpr int kHeadDim = 128;
constexpr int kAttnMaxRep = 8;  // query heads per kv head
constexpr int kAttnUnroll = 4;  // cache rows (K and V each) in flight per half warp (8 with one query head)

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
    __align__(16) float q[kAttnMaxRep][kHeadDim];     // rotated queries times scale * log2(e)
    __align__(16) float red[kAttnWorkers][kHeadDim];  // one query head's partial outputs
    float red_m[kAttnWorkers];
    float red_l[kAttnWorkers];
    float part_m[kAttnMaxRep];  // this block's partials, read by the cluster
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

__device__ __forceinline__ float fast_exp2(float x) {
    float y;
    asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
    return y;
}

// One pass over the cache: every half warp keeps a running (max, sum, weighted V) per query
// head for the positions it visits (16 lanes x 8 dims = one 128-wide row per load), K and V
// rows of kAttnUnroll positions are requested together so that 2 * kAttnUnroll 16-byte loads
// per lane are in flight; the half warps of a block meet in shared memory, the blocks of a
// cluster through distributed shared memory, both in a fixed order.
template <int DT, int REP>
__device__ __forceinline__ void attention_block(const AttnArgs& a, AttnSmem* sm) {
    cg::cluster_group cluster = cg::this_cluster();
    const int S = static_cast<int>(cluster.num_blocks());
    const int rank = static_cast<int>(cluster.block_rank());
    const int hk = blockIdx.y, t = blockIdx.z;
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const int half = lane >> 4, l16 = lane & 15;
    const int worker = 2 * warp + half;
    const int rep = a.q_heads / a.kv_heads;
    const int L = a.pos + 1;
    const int l_lo = static_cast<int>(static_cast<int64_t>(rank) * L / S);
    const int l_hi = static_cast<int>(static_cast<int64_t>(rank + 1) * L / S);
    const float qscale = rsqrtf(static_cast<float>(kHeadDim)) * 1.4426950408889634f;
    const uint32_t half_mask = 0xFFFFu << (16 * half);  // the two halves of a warp work on different keys

    AFX_TRACE_REGION(0);
    AFX_MARK(0);
    uint16_t* kc = a.k_cache + static_cast<size_t>(t) * a.max_seq * a.kv_heads * kHeadDim;
    uint16_t* vc = a.v_cache + static_cast<size_t>(t) * a.max_seq * a.kv_heads * kHeadDim;
    // With one query head per kv head the registers allow it: the past rows of this half
    // warp's first batch were written by earlier tokens' attention kernels -- at least one
    // layer step (five grids) back, so complete by the ordering rule stated in fused_op_block
    // -- and are requested before the wait for q, k, v.
    constexpr int U = REP == 1 ? 2 * kAttnUnroll : kAttnUnroll;
    constexpr bool kEarly = REP == 1;
    uint4 kraw[U], vraw[U];
    if (kEarly) {
        const size_t rs = static_cast<size_t>(a.kv_heads) * kHeadDim;
        const size_t ho = static_cast<size_t>(hk) * kHeadDim + l16 * 8;
#pragma unroll
        for (int u = 0; u < U; ++u) {
            const int p = l_lo + worker + u * kAttnWorkers;
            if (p < l_hi && p < a.pos) {
                kraw[u] = *reinterpret_cast<const uint4*>(kc + static_cast<size_t>(p) * rs + ho);
                vraw[u] = *reinterpret_cast<const uint4*>(vc + static_cast<size_t>(p) * rs + ho);
            }
        }
    }
    asm volatile("griddepcontrol.wait;" ::: "memory");
    asm volatile("griddepcontrol.launch_dependents;" ::: "memory");  // only after the wait (see fused_op_block)
    AFX_MARK(1);

    const float* row = a.qkv + static_cast<size_t>(t) * a.n_qkv;
    const float* cs = a.rope_cos + static_cast<size_t>(a.pos) * (kHeadDim / 2);
    const float* sn = a.rope_sin + static_cast<size_t>(a.pos) * (kHeadDim / 2);
    const size_t row_stride = static_cast<size_t>(a.kv_heads) * kHeadDim;
    const size_t head_off = static_cast<size_t>(hk) * kHeadDim + l16 * 8;

    // rotated, pre-scaled queries of this kv head's group
    for (int e = tid; e < rep * (kHeadDim / 2); e += kAttnThreads) {
        const int r = e / (kHeadDim / 2), i = e - r * (kHeadDim / 2);
        const float* qh = row + static_cast<size_t>(hk * rep + r) * kHeadDim;
        const float x0 = qh[2 * i], x1 = qh[2 * i + 1];
        sm->q[r][2 * i] = (x0 * cs[i] - x1 * sn[i]) * qscale;
        sm->q[r][2 * i + 1] = (x0 * sn[i] + x1 * cs[i]) * qscale;
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

    float m_run[REP], l_run[REP], acc[REP][8];
#pragma unroll
    for (int r = 0; r < REP; ++r) {
        m_run[r] = -INFINITY;
        l_run[r] = 0.0f;
#pragma unroll
        for (int j = 0; j < 8; ++j) acc[r][j] = 0.0f;
    }

    // rows of a batch that are not in registers yet: all of them, or (first batch, requested
    // before the wait) only the row this kernel has just appended
    auto fetch = [&](int p0, bool only_new) {
#pragma unroll
        for (int u = 0; u < U; ++u) {
            const int p = p0 + u * kAttnWorkers;
            if (p < l_hi && (!only_new || p >= a.pos)) {
                kraw[u] = *reinterpret_cast<const uint4*>(kc + static_cast<size_t>(p) * row_stride + head_off);
                vraw[u] = *reinterpret_cast<const uint4*>(vc + static_cast<size_t>(p) * row_stride + head_off);
            }
        }
    };
    AFX_MARK(2);
    fetch(l_lo + worker, kEarly);
    for (int p0 = l_lo + worker; p0 < l_hi; p0 += kAttnWorkers * U) {
        float sc[REP][U];
#pragma unroll
        for (int r = 0; r < REP; ++r) {
            if (r < rep) {
                const float4 qa = *reinterpret_cast<const float4*>(&sm->q[r][l16 * 8]);
                const float4 qb = *reinterpret_cast<const float4*>(&sm->q[r][l16 * 8 + 4]);
#pragma unroll
                for (int u = 0; u < U; ++u) {
                    float d = -INFINITY;
                    if (p0 + u * kAttnWorkers < l_hi) {  // uniform over the half warp
                        float kv[8];
                        unpack8_f16(kraw[u], kv);
                        d = qa.x * kv[0];
                        d = fmaf(qa.y, kv[1], d);
                        d = fmaf(qa.z, kv[2], d);
                        d = fmaf(qa.w, kv[3], d);
                        d = fmaf(qb.x, kv[4], d);
                        d = fmaf(qb.y, kv[5], d);
                        d = fmaf(qb.z, kv[6], d);
                        d = fmaf(qb.w, kv[7], d);
                        d += __shfl_xor_sync(half_mask, d, 8);
                        d += __shfl_xor_sync(half_mask, d, 4);
                        d += __shfl_xor_sync(half_mask, d, 2);
                        d += __shfl_xor_sync(half_mask, d, 1);
                    }
                    sc[r][u] = d;
                }
            }
        }
#pragma unroll
        for (int r = 0; r < REP; ++r) {
            if (r < rep) {
                float mn = m_run[r];
#pragma unroll
                for (int u = 0; u < U; ++u) mn = fmaxf(mn, sc[r][u]);
                const float f = fast_exp2(m_run[r] - mn);  // 0 on the first visit (m_run = -inf)
                m_run[r] = mn;
                l_run[r] *= f;
#pragma unroll
                for (int j = 0; j < 8; ++j) acc[r][j] *= f;
#pragma unroll
                for (int u = 0; u < U; ++u) {
                    if (p0 + u * kAttnWorkers < l_hi) {
                        const float pw = fast_exp2(sc[r][u] - mn);
                        l_run[r] += pw;
                        float vv[8];
                        unpack8_f16(vraw[u], vv);
#pragma unroll
                        for (int j = 0; j < 8; ++j) acc[r][j] = fmaf(pw, vv[j], acc[r][j]);
                    }
                }
            }
        }
        if (p0 + kAttnWorkers * U < l_hi) fetch(p0 + kAttnWorkers * U, false);
    }

    AFX_MARK(3);
    // meet the half warps of the block (fixed order), one query head at a time
#pragma unroll
    for (int r = 0; r < REP; ++r) {
        if (r < rep) {
            float4* dst = reinterpret_cast<float4*>(&sm->red[worker][l16 * 8]);
            dst[0] = make_float4(acc[r][0], acc[r][1], acc[r][2], acc[r][3]);
            dst[1] = make_float4(acc[r][4], acc[r][5], acc[r][6], acc[r][7]);
            if (l16 == 0) {
                sm->red_m[worker] = m_run[r];
                sm->red_l[worker] = l_run[r];
            }
            __syncthreads();
            if (tid <= kHeadDim) {
                float M = -INFINITY;
#pragma unroll
                for (int g = 0; g < kAttnWorkers; ++g) M = fmaxf(M, sm->red_m[g]);
                float s = 0.0f;
#pragma unroll
                for (int g = 0; g < kAttnWorkers; ++g) {
                    // a half warp that saw no position has m = -inf, l = 0, acc = 0
                    const float w = sm->red_m[g] == -INFINITY ? 0.0f : fast_exp2(sm->red_m[g] - M);
                    s = fmaf(w, tid < kHeadDim ? sm->red[g][tid] : sm->red_l[g], s);
                }
                if (tid < kHeadDim) {
                    sm->part_acc[r][tid] = s;
                } else {
                    sm->part_l[r] = s;
                    sm->part_m[r] = M;
                }
            }
            __syncthreads();
        }
    }
    AFX_MARK(4);
    cluster.sync();
    AFX_MARK(5);
    for (int e = rank + S * tid; e < rep * kHeadDim; e += S * kAttnThreads) {
        const int r = e / kHeadDim, d = e - r * kHeadDim;
        // all remote reads first (they are independent), then the merge in block order
        float mq[8], aq[8], lq[8];
#pragma unroll
        for (int q = 0; q < 8; ++q) {
            mq[q] = -INFINITY;
            aq[q] = 0.0f;
            lq[q] = 0.0f;
            if (q < S) {
                mq[q] = cluster.map_shared_rank(&sm->part_m[0], q)[r];
                aq[q] = cluster.map_shared_rank(&sm->part_acc[0][0], q)[r * kHeadDim + d];
                lq[q] = cluster.map_shared_rank(&sm->part_l[0], q)[r];
            }
        }
        float M = -INFINITY;
#pragma unroll
        for (int q = 0; q < 8; ++q) M = fmaxf(M, mq[q]);
        float num = 0.0f, den = 0.0f;
#pragma unroll
        for (int q = 0; q < 8; ++q) {
            const float w = mq[q] == -INFINITY ? 0.0f : fast_exp2(mq[q] - M);
            num = fmaf(w, aq[q], num);
            den = fmaf(w, lq[q], den);
        }
        a.out[static_cast<size_t>(t) * a.q_heads * kHeadDim + static_cast<size_t>(hk * rep + r) * kHeadDim + d] =
            float_to_bits<DT>(num / den);
    }
    AFX_MARK(6);
    cluster.sync();
    AFX_MARK(7);
}

}  // namespace afx
