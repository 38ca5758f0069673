// One sparse operator of a decoder layer as a single kernel: input stage (optional RMSNorm),
// active-channel selection, sparse GEMV, epilogue.  Every block repeats the cheap, exact
// input stage and selection on its own (the activation vector is a few KB and L2 resident),
// so nothing but the previous kernel's output stands between two operators: no separate
// selection launch, no count/index round trips through global memory.
#pragma once

// (the several-token instantiations leave fused_op_block before its one-token streaming loop)
#pragma nv_diag_suppress 128

#include "afx_gemv.cuh"
#include "afx_mma.cuh"
#include "afx_q4.cuh"
#include "afx_select.cuh"

namespace afx {

enum { IN_X = 0, IN_NORM = 1 };

constexpr int kFusedMtRows = 64;  // channels per pipeline stage of the several-token operator

struct FusedArgs {
    const uint16_t* Wt;
    // mixture of experts: if wt_table is given, the weights are wt_table[*wt_sel] (both DEVICE;
    // the choice is made on the device by the router kernel earlier in the stream)
    const uint16_t* const* wt_table;
    const int32_t* wt_sel;
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
    // ---- top-k search hint (may be NULL): 0x10000 | k-th key of this operator's last top-k
    // selection with T == 1; read before the selection, rewritten after it by block (0,0) ----
    int32_t* kth_slot;
    // ---- the same for several tokens (T > 1; may be NULL): T consecutive slots, one per token ----
    int32_t* kth_multi;
    // ---- set by the launcher (several-token operators): column tiles per cluster, 0 or 1 = one ----
    int tiles_per_cluster;
    // ---- set by the launcher: 1 if the grid has one more cluster than column tiles; its block 0
    // repeats input stage and selection only to write the side outputs, off the path of the
    // clusters that stream (its other blocks leave at once) ----
    int side_cluster;
    // ---- several operators of one family in one grid (groups > 1; no side outputs): the
    // column tiles are `groups` equal runs, run g being an operator of the same shape with
    // weights wt_table[wt_sel[g]], input x + g * x_stride, outputs ep.y / ep.out_bits +
    // g * out_stride (elements) and factor ep.scale[g].  Every cluster selects on its run's input. ----
    int groups;
    int64_t x_stride, out_stride;
};

// Dynamic shared memory: [16-bit inputs: T tokens (IN_NORM) or one token (IN_X), each padded
// to a multiple of 8 elements] [T bitmaps of ceil(K/32) flag words, each padded to 16 bytes: where
// the blocks of a cluster exchange the per-token sets they decided] [work area: the key
// histogram during the selection, then the GEMV staging and reduction buffers].
__host__ __device__ inline size_t fused_input_smem(int in_kind, int K, int T) {
    const size_t Kp = (static_cast<size_t>(K) + 7) / 8 * 8;
    return (in_kind == IN_NORM ? static_cast<size_t>(T) : 1) * Kp * 2;
}
__host__ __device__ inline size_t fused_flag_smem(int K, int T = 1) {
    return static_cast<size_t>(T) * ((static_cast<size_t>((K + 31) / 32) * 4 + 15) / 16 * 16);
}
// work = bytes of the work area: the key histogram, or more where the streaming stage needs more
__host__ __device__ inline size_t fused_dyn_smem(int in_kind, int K, int T, size_t work = kKeyHistBytes) {
    return fused_input_smem(in_kind, K, T) + fused_flag_smem(K, T) + (work > kKeyHistBytes ? work : kKeyHistBytes);
}

// GRP: the grid may hold several operators of one family (FusedArgs::groups).
// WMT > 0: several tokens, the streaming stage runs on the tensor cores (afx_mma.cuh) with WMT
// pipeline stages: PW = 256, the work area holds an MtSmem<CAP, WMT> once the selection is over.
// WQ4: the weights are 4-bit rows (afx_sparse_gemv_q4's layout; one token): Wt points at them,
// ldw is the row stride in units of 2 bytes, the tile is PW = 512, 256 or 128 outputs wide and
// the streaming loop and the reduction are the 4-bit kernel's.
template <int DT, int TMAX, int PW, int CAP, int IN, int EP, bool WQ4 = false, bool GRP = false, int WMT = 0>
__device__ __forceinline__ void fused_op_block(const FusedArgs& a, unsigned char* dyn, SelectScratch* sel,
                                               GemvRecv<TMAX>* recv) {
    constexpr int LPC = WQ4 ? PW / kQ4Opl : PW / 8;
    static_assert(WMT > 0 || sizeof(GemvSmem<TMAX, CAP>) <= kKeyHistBytes, "work area too small");
    static_assert(!WQ4 || (TMAX == 1 && CAP * 8 + (kQ4Warps + 1) * PW * 4 <= kKeyHistBytes), "4-bit: one token, sums behind the staged list");
    const int tid = threadIdx.x;
    const int lane = tid & 31;
    const int warp = tid >> 5;
    // CS blocks form a cluster; S of them split the active list of one column tile.  CS == S
    // except for several-token operators with few tiles: there a cluster covers CS / S adjacent
    // tiles, so that more blocks share the per-token selections (a.tiles_per_cluster).
    const int CS = gridDim.x, cs = blockIdx.x;
    const int tpc = (WMT > 0 && a.tiles_per_cluster > 1) ? a.tiles_per_cluster : 1;
    const int S = tpc > 1 ? CS / tpc : CS, s = tpc > 1 ? cs % S : cs;
    const int T = a.T, K = a.K;
    const bool side = a.side_cluster != 0 && blockIdx.y == gridDim.y - 1;  // the cluster without a tile
    int tile = tpc > 1 ? blockIdx.y * tpc + cs / S : blockIdx.y, grp = 0;
    if (GRP && a.groups > 1) {  // (never together with a side cluster)
        const int per = gridDim.y / a.groups;
        grp = tile / per;
        tile -= grp * per;
    }
    auto x_of_run = [&]() { return GRP ? a.x + grp * a.x_stride : a.x; };
    if (side && blockIdx.x != 0) return;  // (a block that has left no longer holds back the next grid)
    // writes the side outputs: block 0 of the side cluster, else block (0,0) next to its GEMV work
    const bool scribe = a.side_cluster != 0 ? side : (blockIdx.x == 0 && blockIdx.y == 0);
    const int nwords = (K + 31) >> 5;

    const int Kp = (K + 7) & ~7;
    uint16_t* xs = reinterpret_cast<uint16_t*>(dyn);
    unsigned char* work = dyn + fused_input_smem(IN, K, T) + fused_flag_smem(K, T);
    uint32_t* hist = reinterpret_cast<uint32_t*>(work);
    GemvSmem<TMAX, CAP>* sm = reinterpret_cast<GemvSmem<TMAX, CAP>*>(work);
    float* red16 = reinterpret_cast<float*>(sel->hist);  // block reduction of the norm

    const uint32_t ld16 = static_cast<uint32_t>(a.ldw >> 3);  // row stride in 16-byte units (the launcher checked the range)
    const bool own = (a.idx_in == nullptr);
    const bool topk = own && a.mode == AFX_MODE_TOPK && a.k > 0 && a.k < K;
    // kernel kinds of a decode step: 1 q|k|v, 2 gate|up, 3 down (the wider plain input), 4 o
    AFX_TRACE_REGION(IN == IN_NORM ? (EP == EP_SILU ? 2 : 1) : (K > a.N ? 3 : 4));
    AFX_MARK(0);
    if (!side) cluster_arrive();  // the side cluster never meets
    if (topk) block_clear_key_hist<kGemvThreads>(hist);  // does not depend on the previous kernel

    // Ordering rule of every kernel of this library: a grid lets its successor be scheduled
    // only AFTER its own dependency wait.  When a grid runs its prologue, its predecessor has
    // therefore passed its wait, i.e. the grid before that one is complete: whatever is read
    // before the wait below must have been written at least two grids earlier (weights and
    // gains: never; the search hint and the predicted set: by the same operator of an earlier
    // token or layer, at least five grids back).
    // the norm's gains are weights: they can be on their way before the wait for h
    constexpr int NH = 4;  // float4 pieces of h (and of the gain) a thread keeps in registers
    float4 gv[NH];
    if (IN == IN_NORM) {
#pragma unroll
        for (int i = 0; i < NH; ++i) {
            const int c = tid + i * kGemvThreads;
            gv[i] = c < (K >> 2) ? reinterpret_cast<const float4*>(a.gain)[c] : make_float4(0.0f, 0.0f, 0.0f, 0.0f);
        }
    }
    // the hint was written by an earlier token's launch of this operator (a launch that reads
    // the value its own scribe block has just rewritten only gets a better hint: the
    // selection's result does not depend on it)
    uint32_t hint = kNoKeyHint;
    if (topk && T == 1 && a.kth_slot != nullptr) {
        const uint32_t v = static_cast<uint32_t>(__ldcg(a.kth_slot));
        if (v & 0x10000u) hint = v & 0x7FFFu;
    }
    uint32_t hint_t[TMAX];  // several tokens: one hint each
#pragma unroll
    for (int t = 0; t < TMAX; ++t) {
        hint_t[t] = kNoKeyHint;
        if (TMAX > 1 && topk && T > 1 && t < T && a.kth_multi != nullptr) {
            const uint32_t v = static_cast<uint32_t>(__ldcg(a.kth_multi + t));
            if (v & 0x10000u) hint_t[t] = v & 0x7FFFu;
        }
    }
    // likewise the predicted set this selection is compared with: the same operator of the
    // predictor layer wrote it, at least one layer (five grids) ago (byte v = the flags of the
    // v-th chunk this thread owns, like `fl`)
    unsigned long long pm = 0ull;
    if (scribe && own && a.bitmap_pred != nullptr) {
        int q_lo, q_hi;
        thread_chunk_range(K, q_lo, q_hi);
        const uint8_t* pred = reinterpret_cast<const uint8_t*>(a.bitmap_pred);
        for (int c = q_lo; c < q_hi; ++c) pm |= static_cast<unsigned long long>(__ldcg(pred + c)) << (8 * (c - q_lo));
    }
    asm volatile("griddepcontrol.wait;" ::: "memory");
    asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
    AFX_MARK(1);

    // ---- input stage --------------------------------------------------------------------
    if (IN == IN_NORM) {
        // x = round(h / rms(h) * gain), every block for itself (K % 8 == 0, 16-byte aligned rows)
        const int nq = K >> 2;
        for (int t = 0; t < T; ++t) {
            const float4* ht = reinterpret_cast<const float4*>(a.h + static_cast<size_t>(t) * K);
            float4 hv[NH];
            float ss = 0.0f;
#pragma unroll
            for (int i = 0; i < NH; ++i) {
                const int c = tid + i * kGemvThreads;
                hv[i] = c < nq ? ht[c] : make_float4(0.0f, 0.0f, 0.0f, 0.0f);
                ss = fmaf(hv[i].x, hv[i].x, ss);
                ss = fmaf(hv[i].y, hv[i].y, ss);
                ss = fmaf(hv[i].z, hv[i].z, ss);
                ss = fmaf(hv[i].w, hv[i].w, ss);
            }
            for (int c = tid + NH * kGemvThreads; c < nq; c += kGemvThreads) {
                const float4 v = ht[c];
                ss = fmaf(v.x, v.x, ss);
                ss = fmaf(v.y, v.y, ss);
                ss = fmaf(v.z, v.z, ss);
                ss = fmaf(v.w, v.w, ss);
            }
            ss = warp_sum(ss);
            if (t > 0) __syncthreads();  // the previous token's sums have been read
            if (lane == 0) red16[warp] = ss;
            __syncthreads();
            float tot = 0.0f;  // the 16 warp sums in warp order, read four at a time
#pragma unroll
            for (int w = 0; w < kGemvWarps; w += 4) {
                const float4 v = *reinterpret_cast<const float4*>(red16 + w);
                tot += v.x;
                tot += v.y;
                tot += v.z;
                tot += v.w;
            }
            const float inv = 1.0f / sqrtf(tot / static_cast<float>(K) + a.eps);
            const float4* gq = reinterpret_cast<const float4*>(a.gain);
            auto emit = [&](int c, const float4& v, const float4& g) {
                const uint32_t lo = static_cast<uint32_t>(float_to_bits<DT>(v.x * inv * g.x)) |
                                    (static_cast<uint32_t>(float_to_bits<DT>(v.y * inv * g.y)) << 16);
                const uint32_t hi = static_cast<uint32_t>(float_to_bits<DT>(v.z * inv * g.z)) |
                                    (static_cast<uint32_t>(float_to_bits<DT>(v.w * inv * g.w)) << 16);
                reinterpret_cast<uint2*>(xs + static_cast<size_t>(t) * Kp)[c] = make_uint2(lo, hi);
                if (scribe && a.xnorm_out != nullptr)
                    reinterpret_cast<uint2*>(a.xnorm_out + static_cast<size_t>(t) * K)[c] = make_uint2(lo, hi);
            };
#pragma unroll
            for (int i = 0; i < NH; ++i) {
                const int c = tid + i * kGemvThreads;
                if (c < nq) emit(c, hv[i], gv[i]);
            }
            for (int c = tid + NH * kGemvThreads; c < nq; c += kGemvThreads) emit(c, ht[c], gq[c]);
        }
        __syncthreads();
    }
    // 16-bit input of token t, channel j, once the stage above / below has run
    auto x_at = [&](int t, int j) -> uint16_t {
        if (IN == IN_NORM) return xs[static_cast<size_t>(t) * Kp + j];
        return T == 1 ? xs[j] : x_of_run()[static_cast<size_t>(t) * K + j];
    };
    AFX_MARK(2);

    // ---- selection ----------------------------------------------------------------------
    int cnt = 0;
    int pos0 = 0;                  // list position of this thread's first active channel
    unsigned long long fl = 0ull;  // this thread's active flags (own selection)
    const int out0 = tile * PW + (lane % LPC) * (WQ4 ? kQ4Opl : 8);
    const bool lane_ok = out0 < a.N;
    // One token, top-k: the list length is k whatever x holds, so this block's part
    // [c_lo, c_hi) of the list is known before the selection and the pass that decides the
    // flags (it has the channel's bits in registers) stages the first CAP entries directly.
    const bool early = topk && T == 1;
    // one word per chunk, in the work area behind the staging and reduction buffers
    constexpr size_t kXchgOffset = kKeyHistBytes - (kSelectFastMaxK / 8) * 4;
    constexpr bool kXchgFits = sizeof(GemvSmem<TMAX, CAP>) <= kXchgOffset;
    static_assert(TMAX > 1 || kXchgFits, "work area too small for the chunk exchange");
    uint32_t* xchg = kXchgFits ? reinterpret_cast<uint32_t*>(work + kXchgOffset) : nullptr;
    bool first_staged = false;
    // Several tokens: the blocks of a cluster share the work -- block s decides the sets of the
    // tokens t with t % CS == cs and writes their flags into every block's table of per-token
    // bitmaps (distributed shared memory); after one cluster barrier every thread reads the
    // union for its own chunks.  (The side cluster works alone and decides every token.)
    const bool share = TMAX > 1 && T > 1 && own && !side && CS > 1;
    uint8_t* const ftab = dyn + fused_input_smem(IN, K, T);
    const size_t fstride = fused_flag_smem(K);
    if (own) {
        const int e_lo = s * a.k / S, e_n = min(CAP, (s + 1) * a.k / S - e_lo);
        if (share) cluster_wait();  // pairs with the cluster_arrive() at kernel start: the peers are running
        bool first = true;
        for (int t = 0; t < T; ++t) {
            if (share && t % CS != cs) continue;
            const uint16_t* xt = xs + (IN == IN_NORM ? static_cast<size_t>(t) * Kp : 0);
            if (IN == IN_X) {
                if (!first) __syncthreads();  // the previous token's keys are still being read
                block_stage_token(x_of_run() + static_cast<size_t>(t) * K, K, xs);
            }
            if (early) {
                fl |= block_token_flags<DT, kGemvThreads>(
                    xt, K, a.mode, a.k, a.tau, hist, first, sel, true, pos0, cnt, [&](int j, int pos, uint16_t bits) {
                        const int p = pos - e_lo;
                        if (p >= 0 && p < e_n) {  // the histogram is dead by now: its memory is the staging area
                            sm->col[p] = static_cast<uint32_t>(j) * ld16;
                            sm->xv[0][p] = bits_to_float<DT>(bits);
                        }
                    }, e_lo, e_lo + e_n, hint, xchg);
                first_staged = true;
                if (scribe && tid == 0 && a.kth_slot != nullptr) *a.kth_slot = 0x10000 | sel->res[0];
            } else {
                uint32_t thr_t = 0;
                uint32_t h_t = kNoKeyHint;
#pragma unroll
                for (int u = 0; u < TMAX; ++u)
                    if (u == t) h_t = hint_t[u];
                const unsigned long long ft =
                    block_token_flags<DT, kGemvThreads>(xt, K, a.mode, a.k, a.tau, hist, first, sel, T == 1, pos0, cnt,
                                                        NoEmit(), 0, 0x7FFFFFFF, h_t, nullptr, &thr_t);
                if (scribe && tid == 0 && topk && T > 1 && a.kth_multi != nullptr) a.kth_multi[t] = 0x10000 | thr_t;
                if (share) {
                    int q_lo, q_hi;
                    thread_chunk_range(K, q_lo, q_hi);
                    for (int q = 0; q < CS; ++q) {
                        uint8_t* dst = cg::this_cluster().map_shared_rank(ftab + static_cast<size_t>(t) * fstride, q);
                        for (int c = q_lo; c < q_hi; ++c) dst[c] = static_cast<uint8_t>(ft >> (8 * (c - q_lo)));
                    }
                } else {
                    fl |= ft;
                }
            }
            first = false;
        }
        if (share) {
            cluster_arrive();  // the flags written above are visible to the peers after their wait
            cluster_wait();
            int q_lo, q_hi;
            thread_chunk_range(K, q_lo, q_hi);
            for (int t = 0; t < T; ++t)
                for (int c = q_lo; c < q_hi; ++c)
                    fl |= static_cast<unsigned long long>(ftab[static_cast<size_t>(t) * fstride + c]) << (8 * (c - q_lo));
        }
        if (T > 1) pos0 = block_prefix(__popcll(fl), sel->wtot[2], cnt);
    } else {
        if (IN == IN_X && T == 1) block_stage_token(x_of_run(), K, xs);
        cnt = *a.count_in;
        cnt = max(0, min(cnt, K));
    }
    // ---- side outputs (one block of the grid): plain stores that drain while the block streams ----
    if (scribe) {
        if (own) {
            if (a.idx_out != nullptr) for_each_owned_active(fl, K, pos0, [&](int j, int pos) { a.idx_out[pos] = j; });
            int q_lo, q_hi;
            thread_chunk_range(K, q_lo, q_hi);
            if (a.bitmap_out != nullptr) {  // byte c of the bitmap = the flags of chunk c
                uint8_t* bytes = reinterpret_cast<uint8_t*>(a.bitmap_out);
                for (int c = q_lo; c < q_hi; ++c) bytes[c] = static_cast<uint8_t>(fl >> (8 * (c - q_lo)));
                for (int c = ((K + 7) >> 3) + tid; c < nwords * 4; c += kGemvThreads) bytes[c] = 0;
            }
            if (a.bitmap_pred != nullptr) {
                // A \ P in ascending order, |A & P|
                const unsigned long long ms = fl & ~pm;
                int n_miss;
                const int m0 = block_prefix(__popcll(ms), sel->wtot[3], n_miss);
                if (a.miss_out != nullptr)
                    for_each_owned_active(ms, K, m0, [&](int j, int pos) { a.miss_out[pos] = j; });
                if (tid == 0) {
                    if (a.miss_count != nullptr) *a.miss_count = n_miss;
                    if (a.hit_count != nullptr) *a.hit_count = cnt - n_miss;
                }
            }
        } else if (a.idx_out != nullptr && a.idx_out != a.idx_in) {
            for (int i = tid; i < cnt; i += kGemvThreads) a.idx_out[i] = a.idx_in[i];
        }
        if (tid == 0 && a.count_out != nullptr) *a.count_out = cnt;
        if (side) return;
    }
    AFX_MARK(3);
    const uint16_t* Wt = a.wt_table != nullptr ? a.wt_table[a.wt_sel[GRP ? grp : 0]] : a.Wt;
    const int c_lo = s * cnt / S;  // S <= 8, cnt <= 2^20: no overflow
    const int c_hi = (s + 1) * cnt / S;

    float acc[TMAX][8];
#pragma unroll
    for (int t = 0; t < TMAX; ++t)
#pragma unroll
        for (int q = 0; q < 8; ++q) acc[t][q] = 0.0f;
    f32x2 qacc[8];  // 4-bit weights: 16 outputs per lane
#pragma unroll
    for (int i = 0; i < 8; ++i) qacc[i] = pack_f32x2(0.0f, 0.0f);

    const int n_mine = __popcll(fl);
    if (WMT) {
        using MtT = MtSmem<CAP, (WMT > 0 ? WMT : 2), kFusedMtRows>;
        MtT* mt = reinterpret_cast<MtT*>(work);
        constexpr int kMtCap = CAP;
        float c4[4] = {0.0f, 0.0f, 0.0f, 0.0f};
        const uint4* wtile16 = reinterpret_cast<const uint4*>(Wt + static_cast<size_t>(tile) * kMtTile);
        const int n_chunks = max(0, min(kMtTile, a.N - tile * kMtTile)) >> 3;
        // (the last cluster of a grid with several tiles per cluster may hold a block without a
        // tile: it only shares the selections and meets the barriers)
        for (int c0 = c_lo; n_chunks > 0 && c0 < c_hi; c0 += kMtCap) {
            const int staged = min(kMtCap, c_hi - c0);
            __syncthreads();  // the work area is free: the histogram / the previous pass has been read
            if (own) {
                if (pos0 < c0 + staged && pos0 + n_mine > c0) {
                    for_each_owned_active(fl, K, pos0, [&](int j, int pos) {
                        const int p = pos - c0;
                        if (p >= 0 && p < staged) {
                            mt->col[p] = static_cast<uint32_t>(j) * ld16;
#pragma unroll
                            for (int t = 0; t < TMAX; ++t)
                                if (t < T) mt->xb[t][p] = x_at(t, j);
                        }
                    });
                }
            } else {
                for (int i = tid; i < staged; i += kGemvThreads) {
                    const int j = a.idx_in[c0 + i];
                    mt->col[i] = static_cast<uint32_t>(j) * ld16;
#pragma unroll
                    for (int t = 0; t < TMAX; ++t)
                        if (t < T) mt->xb[t][i] = x_at(t, j);
                }
            }
            mt_pad_inputs(mt, T, staged);
            __syncthreads();
            mt_stream_pass<DT>(wtile16, mt, staged, n_chunks, c4);
        }
        EpilogueArgs ep = a.ep;
        if (!share) cluster_wait();  // pairs with the cluster_arrive() at kernel start
        mt_finish<DT>(c4, mt, T, tile, a.N, EP, ep, S, s, cs - s);
        return;
    }
    for (int c0 = c_lo; c0 < c_hi; c0 += CAP) {
        const int staged = min(CAP, c_hi - c0);
        if (!(first_staged && c0 == c_lo)) {
            __syncthreads();  // the work area is free: the histogram / the previous stage has been read
            // ---- stage (column, x values) of list positions [c0, c0 + staged) ----
            if (own) {
                if (pos0 < c0 + staged && pos0 + n_mine > c0) {
                    for_each_owned_active(fl, K, pos0, [&](int j, int pos) {
                        const int p = pos - c0;
                        if (p >= 0 && p < staged) {
                            sm->col[p] = static_cast<uint32_t>(j) * ld16;
#pragma unroll
                            for (int t = 0; t < TMAX; ++t)
                                if (t < T) sm->xv[t][p] = bits_to_float<DT>(x_at(t, j));
                        }
                    });
                }
            } else {
                for (int i = tid; i < staged; i += kGemvThreads) {
                    const int j = a.idx_in[c0 + i];
                    sm->col[i] = static_cast<uint32_t>(j) * ld16;
#pragma unroll
                    for (int t = 0; t < TMAX; ++t)
                        if (t < T) sm->xv[t][i] = bits_to_float<DT>(x_at(t, j));
                }
            }
        }
        __syncthreads();
        AFX_MARK(4);
        if (WQ4) {
            if (lane_ok)
                q4_stream<LPC>(reinterpret_cast<const unsigned char*>(Wt), a.N, out0 / kQ4Opl, sm->col, sm->xv[0], staged, qacc);
        } else if (lane_ok) {
            gemv_stream<DT, TMAX, PW, CAP, false>(reinterpret_cast<const uint4*>(Wt + out0), T, sm, staged, acc);
        }
    }
    AFX_MARK(5);

    AFX_MARK(6);

    EpilogueArgs ep = a.ep;
    if (GRP && a.groups > 1) {
        if (ep.y != nullptr) ep.y += grp * a.out_stride;
        if (ep.out_bits != nullptr) ep.out_bits += grp * a.out_stride;
        if (ep.scale != nullptr) ep.scale += grp;
    }
    if (WQ4) {
        cluster_wait();  // pairs with the cluster_arrive() at kernel start
        q4_finish<DT, LPC>(qacc, reinterpret_cast<float*>(work) + 2 * CAP, tile, a.N,
                           EP == EP_SILU ? Q4_SILU : (EP == EP_ACCUM ? Q4_ACCUM : Q4_STORE), ep.y, ep.out_bits);
    } else {
        gemv_finish_tile<DT, TMAX, PW, CAP, EP>(acc, T, tile, sm, recv, ep, !share);
    }
    AFX_MARK(7);
}

}  // namespace afx
