// One sparse operator of a decoder layer as a single kernel: input stage (optional RMSNorm),
// active-channel selection, sparse GEMV, epilogue.  Every block repeats the cheap, exact
// input stage and selection on its own (the activation vector is a few KB and L2 resident),
// so nothing but the previous kernel's output stands between two operators: no separate
// selection launch, no count/index round trips through global memory.
#pragma once

#include "afx_gemv.cuh"
#include "afx_select.cuh"

namespace afx {

enum { IN_X = 0, IN_NORM = 1 };

struct FusedArgs {
    const uint16_t* Wt;
    int64_t ldw;
    int K, N, T;
    // ---- input: IN_X reads x; IN_NORM computes x = round(h / rms(h) * gain) ----
    const uint16_t* x;  // [T][K] 16-bit floats
    const float* h;     // [T][K] fp32
    const float* gain;  // [K] fp32
    float eps;
    // ---- selection: own selection, or (idx_in != NULL) a list decided earlier ----
    int mode, k;
    float tau;
    const int32_t* idx_in;
    const int32_t* count_in;
    EpilogueArgs ep;
    // ---- side outputs of block (0,0); each may be NULL ----
    int32_t* idx_out;        // the active list used (capacity K)
    int32_t* count_out;
    uint32_t* bitmap_out;    // the same set as a bitmap (own selection only)
    uint16_t* xnorm_out;     // IN_NORM: the normalised, rounded input [T][K]
    const uint32_t* bitmap_pred;  // cross-layer bookkeeping: predicted set P ...
    int32_t* miss_out;            // ... A \ P ascending (capacity K)
    int32_t* miss_count;
    int32_t* hit_count;           // |A & P|
};

// Dynamic shared memory: [T*K 16-bit inputs (IN_NORM only)] [ceil(K/32) flag words].
__host__ __device__ inline size_t fused_dyn_smem(int in_kind, int K, int T) {
    size_t b = static_cast<size_t>((K + 31) / 32) * 4;
    if (in_kind == IN_NORM) b += (static_cast<size_t>(T) * K * 2 + 15) / 16 * 16;
    return b;
}

template <int DT, int TMAX, int PW, int CAP, int IN, int EP>
__device__ __forceinline__ void fused_op_block(const FusedArgs& a, unsigned char* dyn,
                                               GemvSmem<TMAX, CAP>* sm, SelectScratch* sel) {
    constexpr int LPC = PW / 8;
    const int tid = threadIdx.x;
    const int lane = tid & 31;
    const int warp = tid >> 5;
    const int S = gridDim.x, s = blockIdx.x, tile = blockIdx.y;
    const int T = a.T, K = a.K;
    const bool scribe = (blockIdx.x == 0 && blockIdx.y == 0);  // writes the side outputs
    const int nwords = (K + 31) >> 5;

    uint16_t* xs = reinterpret_cast<uint16_t*>(dyn);
    uint32_t* flags = reinterpret_cast<uint32_t*>(
        dyn + (IN == IN_NORM ? (static_cast<size_t>(T) * K * 2 + 15) / 16 * 16 : 0));

    asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
    asm volatile("griddepcontrol.wait;" ::: "memory");

    // ---- input stage --------------------------------------------------------------------
    const uint16_t* xin = a.x;
    if (IN == IN_NORM) {
        for (int t = 0; t < T; ++t) {
            const float* ht = a.h + static_cast<size_t>(t) * K;
            float ss = 0.0f;
            for (int j = tid; j < K; j += kGemvThreads) {
                const float v = ht[j];
                ss = fmaf(v, v, ss);
            }
            ss = warp_sum(ss);
            __syncthreads();
            if (lane == 0) sm->red[0][warp] = ss;
            __syncthreads();
            float tot = 0.0f;
#pragma unroll
            for (int w = 0; w < kGemvWarps; ++w) tot += sm->red[0][w];
            const float inv = 1.0f / sqrtf(tot / static_cast<float>(K) + a.eps);
            for (int j = tid; j < K; j += kGemvThreads) {
                const uint16_t b = float_to_bits<DT>(ht[j] * inv * a.gain[j]);
                xs[static_cast<size_t>(t) * K + j] = b;
                if (scribe && a.xnorm_out != nullptr) a.xnorm_out[static_cast<size_t>(t) * K + j] = b;
            }
        }
        __syncthreads();
        xin = xs;
    }

    // ---- selection ----------------------------------------------------------------------
    int cnt;
    int warp_base = 0;  // position of this warp's first active channel in the list
    int w0 = 0, w1 = 0;
    const bool own = (a.idx_in == nullptr);
    if (own) {
        block_select_flags<DT>(xin, K, T, a.mode, a.k, a.tau, flags, sel);
        warp_word_range(nwords, w0, w1);
        int c = 0;
        for (int w = w0 + lane; w < w1; w += 32) c += __popc(flags[w]);
        c = warp_sum(c);
        warp_base = block_exclusive_over_warps(c, sel->scan);
        cnt = sel->scan[32];
    } else {
        cnt = *a.count_in;
        cnt = max(0, min(cnt, K));
    }
    const int c_lo = static_cast<int>(static_cast<int64_t>(s) * cnt / S);
    const int c_hi = static_cast<int>(static_cast<int64_t>(s + 1) * cnt / S);
    const int out0 = tile * PW + (lane % LPC) * 8;
    const bool lane_ok = out0 < a.N;
    const uint32_t lt_mask = (1u << lane) - 1u;

    float acc[TMAX][8];
#pragma unroll
    for (int t = 0; t < TMAX; ++t)
#pragma unroll
        for (int q = 0; q < 8; ++q) acc[t][q] = 0.0f;

    for (int c0 = c_lo; c0 < c_hi; c0 += CAP) {
        const int staged = min(CAP, c_hi - c0);
        __syncthreads();
        // ---- stage (column, x values) of list positions [c0, c0 + staged) ----
        if (own) {
            int base = warp_base;
            for (int w = w0; w < w1; ++w) {
                const uint32_t bits = flags[w];
                const int n = __popc(bits);
                if (base + n > c0 && base < c0 + staged && ((bits >> lane) & 1u)) {
                    const int pos = base + __popc(bits & lt_mask) - c0;
                    if (pos >= 0 && pos < staged) {
                        const int j = (w << 5) + lane;
                        sm->col[pos] = j;
#pragma unroll
                        for (int t = 0; t < TMAX; ++t)
                            if (t < T) sm->xv[t][pos] = bits_to_float<DT>(xin[static_cast<size_t>(t) * K + j]);
                    }
                }
                base += n;
            }
        } else {
            for (int i = tid; i < staged; i += kGemvThreads) {
                const int j = a.idx_in[c0 + i];
                sm->col[i] = j;
#pragma unroll
                for (int t = 0; t < TMAX; ++t)
                    if (t < T) sm->xv[t][i] = bits_to_float<DT>(xin[static_cast<size_t>(t) * K + j]);
            }
        }
        __syncthreads();
        if (lane_ok) gemv_stream<DT, TMAX, PW, CAP>(a.Wt + out0, a.ldw, T, sm, staged, acc);
    }

    // ---- side outputs (one block of the grid) ---------------------------------------------
    if (scribe) {
        if (own) {
            if (a.idx_out != nullptr) {
                int base = warp_base;
                for (int w = w0; w < w1; ++w) {
                    const uint32_t bits = flags[w];
                    if ((bits >> lane) & 1u) a.idx_out[base + __popc(bits & lt_mask)] = (w << 5) + lane;
                    base += __popc(bits);
                }
            }
            if (a.bitmap_out != nullptr)
                for (int w = tid; w < nwords; w += kGemvThreads) a.bitmap_out[w] = flags[w];
            if (a.bitmap_pred != nullptr) {
                // A \ P in ascending order, |A & P|
                int c = 0;
                for (int w = w0 + lane; w < w1; w += 32) c += __popc(flags[w] & ~a.bitmap_pred[w]);
                c = warp_sum(c);
                int base = block_exclusive_over_warps(c, sel->scan);
                const int n_miss = sel->scan[32];
                if (a.miss_out != nullptr) {
                    for (int w = w0; w < w1; ++w) {
                        const uint32_t bits = flags[w] & ~a.bitmap_pred[w];
                        if ((bits >> lane) & 1u) a.miss_out[base + __popc(bits & lt_mask)] = (w << 5) + lane;
                        base += __popc(bits);
                    }
                }
                if (tid == 0) {
                    if (a.miss_count != nullptr) *a.miss_count = n_miss;
                    if (a.hit_count != nullptr) *a.hit_count = cnt - n_miss;
                }
            }
        } else if (a.idx_out != nullptr && a.idx_out != a.idx_in) {
            for (int i = tid; i < cnt; i += kGemvThreads) a.idx_out[i] = a.idx_in[i];
        }
        if (tid == 0 && a.count_out != nullptr) *a.count_out = cnt;
    }

    gemv_finish_tile<DT, TMAX, PW, CAP, EP>(acc, T, tile, sm, a.ep);
}

}  // namespace afx
