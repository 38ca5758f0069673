// Block-level active-channel selection: |x| top-k (ties to the lower channel id) or threshold,
// OR-ed over T tokens, then an ordered compaction into an ascending index list.
//
// Fast path (K <= 32768, one token's 16-bit patterns in shared memory).  Every thread owns a
// contiguous run of 8-channel chunks, so "ascending channel id" is "ascending thread id" and
// one block-wide prefix scan orders both the tie-break and the compaction.  Top-k finds the
// k-th largest 15-bit magnitude key in ONE counting pass: a full histogram of the 32768
// possible keys (16-bit counters, 64 KB of shared memory) filled with shared-memory atomics
// -- real-valued activations spread over hundreds of distinct keys, so the atomics rarely
// collide, where a histogram of the high key bits alone would serialise on a few exponent
// bins -- followed by a top-down search: per-warp totals, the warp that holds the k-th key,
// the row, the lane, the counter.
//
// The routines are written for one thread block of 256, 512 or 1024 threads so that the
// stand-alone selection kernel and kernels that need the selection as a prologue can share
// them.  Every routine contains block-wide barriers: all threads of the block call it with
// the same arguments.
#pragma once

#include <type_traits>

#include "afx_common.cuh"

namespace afx {

constexpr int kSelectFastMaxK = 32768;  // keys of one token held in shared memory
constexpr int kKeyHistWords = 16384;    // 32768 16-bit counters
constexpr size_t kKeyHistBytes = static_cast<size_t>(kKeyHistWords) * 4;

struct SelectScratch {
    int wtot[4][32];  // per-warp totals for the ordered scans
    int res[4];       // broadcast of the k-th key search
    __align__(16) int hist[256];  // large-K path; the fused operators borrow it for the norm's reduction
    int scan[33];
};

// Words [w0, w1) of a ceil(K/32)-word bitmap owned by the calling warp (contiguous, so that
// a walk over warps in order visits channels in ascending order).
__device__ __forceinline__ void warp_word_range(int nwords, int& w0, int& w1) {
    const int nw = blockDim.x >> 5;
    const int per = (nwords + nw - 1) / nw;
    w0 = warp_id() * per;
    w1 = min(nwords, w0 + per);
    if (w0 > nwords) w0 = nwords;
}

// Exclusive prefix over the warps of the block of one int per warp (`mine`, same in all
// lanes); `total` receives the block's sum.  One barrier.  `buf` (32 ints of shared memory)
// must not be written again before every warp has passed a later barrier.
__device__ __forceinline__ int warp_prefix(int mine, int* buf, int& total) {
    const int nw = blockDim.x >> 5;
    const int lane = lane_id();
    if (lane == 0) buf[warp_id()] = mine;
    __syncthreads();
    const int v = lane < nw ? buf[lane] : 0;
    int incl = v;
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) {
        const int n = __shfl_up_sync(0xFFFFFFFFu, incl, o);
        if (lane >= o) incl += n;
    }
    total = __shfl_sync(0xFFFFFFFFu, incl, 31);
    return __shfl_sync(0xFFFFFFFFu, incl - v, warp_id());
}

// Exclusive prefix over the THREADS of the block (thread order) of `v`; `total` = block sum.
__device__ __forceinline__ int block_prefix(int v, int* buf, int& total) {
    const int lane = lane_id();
    int incl = v;
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) {
        const int n = __shfl_up_sync(0xFFFFFFFFu, incl, o);
        if (lane >= o) incl += n;
    }
    const int wsum = __shfl_sync(0xFFFFFFFFu, incl, 31);
    return warp_prefix(wsum, buf, total) + incl - v;
}

// The chunks (8 channels each) owned by the calling thread: [c_lo, c_hi), at most 8.
__device__ __forceinline__ void thread_chunk_range(int K, int& c_lo, int& c_hi) {
    const int nchunks = (K + 7) >> 3;
    const int m = (nchunks + blockDim.x - 1) / blockDim.x;
    c_lo = min(static_cast<int>(threadIdx.x) * m, nchunks);
    c_hi = min(c_lo + m, nchunks);
}

__device__ __forceinline__ void chunk_keys(const uint16_t* xs, int c, uint32_t (&key)[8]) {
    const uint4 raw = *reinterpret_cast<const uint4*>(xs + (c << 3));
    const uint32_t r[4] = {raw.x, raw.y, raw.z, raw.w};
#pragma unroll
    for (int i = 0; i < 4; ++i) {
        key[2 * i] = r[i] & 0x7FFFu;
        key[2 * i + 1] = (r[i] >> 16) & 0x7FFFu;
    }
}

// Two 15-bit keys per 32-bit word (bits 15 and 31 clear), compared at once against a key
// replicated in both halves: the result has bit 15 / bit 31 set where the low / high key
// is greater.  (0x8000 | key) - (thr + 1) stays within its 16 bits -- no borrow crosses the
// halves -- and keeps bit 15 exactly when key > thr.
constexpr uint32_t kHalfTops = 0x80008000u;
__device__ __forceinline__ uint32_t swar_pair(uint32_t key) { return key * 0x00010001u; }
__device__ __forceinline__ uint32_t swar_gt(uint32_t keys2, uint32_t thr2_plus1) {
    return ((keys2 | kHalfTops) - thr2_plus1) & kHalfTops;
}

// Sets the key histogram to zero (no barrier).
template <int NT>
__device__ __forceinline__ void block_clear_key_hist(uint32_t* hist) {
    uint4* h4 = reinterpret_cast<uint4*>(hist) + threadIdx.x;
#pragma unroll
    for (int i = 0; i < kKeyHistWords / 4 / NT; ++i) h4[i * NT] = make_uint4(0u, 0u, 0u, 0u);
}

// The k-th largest magnitude key (1 <= k <= K) of xs[0..K) (shared memory, 16-byte aligned,
// readable up to the next multiple of 8 elements).  `hist` is kKeyHistWords words of shared
// memory, all zero and visible on entry (block_clear_key_hist + barrier); it is left dirty.
// Returns the key in `thr`, how many channels with exactly that key belong to the top k in
// `need_eq`, and how many channels have that key in `tot_eq`.  Same values in every thread.
template <int NT>
__device__ __forceinline__ void block_kth_key(const uint16_t* xs, int K, int k, uint32_t* hist,
                                              SelectScratch* s, uint32_t& thr, int& need_eq, int& tot_eq) {
    constexpr int NW = NT / 32;
    constexpr int W = kKeyHistWords / NW;  // histogram words per warp
    constexpr int NR = W / 128;            // rows of 32 lanes x 4 words
    static_assert(NR >= 1 && NR * 128 * NW == kKeyHistWords, "block size must be 256, 512 or 1024");
    const int lane = lane_id();
    const int warp = warp_id();
    int c_lo, c_hi;
    thread_chunk_range(K, c_lo, c_hi);
    for (int c = c_lo; c < c_hi; ++c) {
        const uint4 raw = *reinterpret_cast<const uint4*>(xs + (c << 3));
        const uint32_t r[4] = {raw.x, raw.y, raw.z, raw.w};
        const int nvalid = K - (c << 3);  // < 8 only in the last chunk of a K that is no multiple of 8
#pragma unroll
        for (int i = 0; i < 4; ++i) {
            const uint32_t k0 = r[i] & 0x7FFFu, k1 = (r[i] >> 16) & 0x7FFFu;
            if (2 * i < nvalid) atomicAdd(&hist[k0 >> 1], (k0 & 1u) ? 0x10000u : 1u);
            if (2 * i + 1 < nvalid) atomicAdd(&hist[k1 >> 1], (k1 & 1u) ? 0x10000u : 1u);
        }
    }
    __syncthreads();
    // counters of this warp's slice, highest keys last: row i, lane l holds words
    // warp*W + (i*32 + l)*4 .. +4
    const uint32_t* mine = hist + warp * W + lane * 4;
    uint32_t packed = 0;  // two 16-bit sums, neither overflows (K <= 32768)
#pragma unroll
    for (int i = 0; i < NR; ++i) {
        const uint4 v = *reinterpret_cast<const uint4*>(mine + i * 128);
        packed += v.x + v.y + v.z + v.w;
    }
    const int lane_total = static_cast<int>((packed & 0xFFFFu) + (packed >> 16));
    const int warp_total = __reduce_add_sync(0xFFFFFFFFu, lane_total);
    int total;
    const int below = warp_prefix(warp_total, s->wtot[0], total);
    const int above = total - below - warp_total;  // keys in the slices of higher warps
    if (above < k && k <= above + warp_total) {    // exactly one warp holds the k-th largest key
        int rem = k - above;                       // rank from the top inside this warp's slice
        int row = 0, row_lane_sum = 0;
        bool found = false;
        int rowsum[NR];
#pragma unroll
        for (int i = 0; i < NR; ++i) {
            const uint4 v = *reinterpret_cast<const uint4*>(mine + i * 128);
            const uint32_t p = v.x + v.y + v.z + v.w;
            rowsum[i] = static_cast<int>((p & 0xFFFFu) + (p >> 16));
        }
#pragma unroll
        for (int i = NR - 1; i >= 0; --i) {
            const int rt = __reduce_add_sync(0xFFFFFFFFu, rowsum[i]);
            if (!found) {
                if (rem <= rt) {
                    found = true;
                    row = i;
                    row_lane_sum = rowsum[i];
                } else {
                    rem -= rt;
                }
            }
        }
        // inclusive suffix sums over the lanes of that row (higher lanes hold higher keys)
        int suf = row_lane_sum;
#pragma unroll
        for (int o = 1; o < 32; o <<= 1) {
            const int n = __shfl_down_sync(0xFFFFFFFFu, suf, o);
            if (lane + o < 32) suf += n;
        }
        const uint32_t ok = __ballot_sync(0xFFFFFFFFu, suf >= rem);
        const int l_star = 31 - __clz(static_cast<int>(ok));
        if (lane == l_star) {
            rem -= suf - row_lane_sum;  // keys in higher lanes of the row
            const uint4 v = *reinterpret_cast<const uint4*>(mine + row * 128);
            const uint32_t w[4] = {v.x, v.y, v.z, v.w};
            const int word0 = warp * W + (row * 32 + lane) * 4;
            bool done = false;
#pragma unroll
            for (int q = 3; q >= 0; --q) {
#pragma unroll
                for (int h = 1; h >= 0; --h) {
                    const int c = static_cast<int>((w[q] >> (16 * h)) & 0xFFFFu);
                    if (!done) {
                        if (rem <= c) {
                            done = true;
                            s->res[0] = 2 * (word0 + q) + h;
                            s->res[1] = rem;
                            s->res[2] = c;
                        } else {
                            rem -= c;
                        }
                    }
                }
            }
        }
    }
    __syncthreads();
    thr = static_cast<uint32_t>(s->res[0]);
    need_eq = s->res[1];
    tot_eq = s->res[2];
}

// Keys searched around a hint of the k-th key: about +-19 % in magnitude for either type.
template <int DT>
struct KeyWindow {
    static constexpr int kBins = DT == AFX_BF16 ? 64 : 512;
};
constexpr uint32_t kNoKeyHint = 0xFFFFFFFFu;

// block_kth_key with a hint (a key near the expected answer, e.g. the one found for the
// previous token): counts the keys above a window of KeyWindow<DT>::kBins keys around the hint
// and histograms only the keys inside it -- two masked compares per word and a few
// uncontended atomics instead of one atomic per key, and one warp resolves the window.
// Exact whenever it returns true; returns false (same value in every thread, outputs
// untouched, `hist` clean again) when the k-th key lies outside the window.  `hist` as for
// block_kth_key; words [0, kBins) are left dirty and may be rewritten only after the block's
// next barrier (the warps read them at their own pace).
template <int DT, int NT>
__device__ __forceinline__ bool block_kth_key_near(const uint16_t* xs, int K, int k, uint32_t hint,
                                                   uint32_t* hist, SelectScratch* s, uint32_t& thr,
                                                   int& need_eq, int& tot_eq) {
    constexpr int WB = KeyWindow<DT>::kBins;
    constexpr int P = WB / 32;  // bins per lane of the resolving warp
    static_assert(P == 2 || P % 4 == 0, "window bins per lane: 2 or a multiple of 4");
    const int lane = lane_id();
    const int lo = max(0, min(static_cast<int>(hint & 0x7FFFu) - WB / 2, 32768 - WB));
    // swar_gt(keys, pair(v)) marks keys >= v (it tests key > v - 1); lo + WB <= 0x8000 keeps
    // the subtraction inside its half
    const uint32_t lo2 = swar_pair(static_cast<uint32_t>(lo)), hi2 = swar_pair(static_cast<uint32_t>(lo + WB));
    int c_lo, c_hi;
    thread_chunk_range(K, c_lo, c_hi);
    int above = 0;
    for (int c = c_lo; c < c_hi; ++c) {
        const uint4 raw = *reinterpret_cast<const uint4*>(xs + (c << 3));
        const uint32_t r[4] = {raw.x & 0x7FFF7FFFu, raw.y & 0x7FFF7FFFu, raw.z & 0x7FFF7FFFu, raw.w & 0x7FFF7FFFu};
        const int nvalid = K - (c << 3);
        uint32_t am = 0;
#pragma unroll
        for (int i = 0; i < 4; ++i) {
            const uint32_t a = swar_gt(r[i], hi2);
            uint32_t in = swar_gt(r[i], lo2) & ~a;
            // the zero padding of a partial last chunk would fall into a window that starts at 0
            if (nvalid < 8) in &= (2 * i < nvalid ? 0x8000u : 0u) | (2 * i + 1 < nvalid ? 0x80000000u : 0u);
            am |= a >> i;
            if (in & 0x8000u) atomicAdd(&hist[(r[i] & 0xFFFFu) - lo], 1u);
            if (in & 0x80000000u) atomicAdd(&hist[(r[i] >> 16) - lo], 1u);
        }
        above += __popc(am);
    }
    AFX_MARK(11);
    above = __reduce_add_sync(0xFFFFFFFFu, above);
    if (lane == 0) s->wtot[0][warp_id()] = above;
    AFX_MARK(12);
    __syncthreads();
    AFX_MARK(13);
    // Every warp resolves the window for itself from the same counters: nothing to broadcast.
    constexpr int NW = NT / 32;
    const int ab = __reduce_add_sync(0xFFFFFFFFu, lane < NW ? s->wtot[0][lane] : 0);
    uint32_t cnt[P];
    if (P == 2) {
        const uint2 v = *reinterpret_cast<const uint2*>(hist + lane * 2);
        cnt[0] = v.x;
        cnt[1] = v.y;
    } else {
#pragma unroll
        for (int q = 0; q < P / 4; ++q) {
            const uint4 v = *reinterpret_cast<const uint4*>(hist + lane * P + q * 4);
            cnt[4 * q] = v.x;
            cnt[4 * q + 1] = v.y;
            cnt[4 * q + 2] = v.z;
            cnt[4 * q + 3] = v.w;
        }
    }
    int lane_sum = 0;
#pragma unroll
    for (int q = 0; q < P; ++q) lane_sum += static_cast<int>(cnt[q]);
    int suf = lane_sum;  // inclusive suffix sums: higher lanes hold higher keys
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) {
        const int n = __shfl_down_sync(0xFFFFFFFFu, suf, o);
        if (lane + o < 32) suf += n;
    }
    const int inside = __shfl_sync(0xFFFFFFFFu, suf, 0);
    if (!(ab < k && k <= ab + inside)) {  // same outcome in every warp
        __syncthreads();                  // every warp has read the window
        for (int i = threadIdx.x; i < WB; i += NT) hist[i] = 0u;
        __syncthreads();
        return false;
    }
    int rem = k - ab;  // rank from the top inside the window
    const uint32_t has = __ballot_sync(0xFFFFFFFFu, suf >= rem);
    const int l_star = 31 - __clz(static_cast<int>(has));
    int my_thr = 0, my_need = 0, my_tot = 0;
    if (lane == l_star) {
        rem -= suf - lane_sum;
        bool done = false;
#pragma unroll
        for (int q = P - 1; q >= 0; --q) {
            const int cq = static_cast<int>(cnt[q]);
            if (!done) {
                if (rem <= cq) {
                    done = true;
                    my_thr = lo + lane * P + q;
                    my_need = rem;
                    my_tot = cq;
                } else {
                    rem -= cq;
                }
            }
        }
        if (warp_id() == 0) s->res[0] = my_thr;  // for the caller that records the key
    }
    thr = static_cast<uint32_t>(__shfl_sync(0xFFFFFFFFu, my_thr, l_star));
    need_eq = __shfl_sync(0xFFFFFFFFu, my_need, l_star);
    tot_eq = __shfl_sync(0xFFFFFFFFu, my_tot, l_star);
    return true;
}

// Active flags of ONE token for the calling thread's chunks: byte v of the result covers the
// 8 channels of chunk c_lo + v (bit e = channel 8 * (c_lo + v) + e).  xs as for
// block_kth_key.  `hist` is the key histogram (top-k only); `hist_clean` says that it is
// already zero and visible.  With `single` set (the token is the only one) the call also
// returns the list position of the thread's first active channel in `pos0` and the length
// of the list in `cnt`, from the same scan that orders the tie-break, and calls
// emit(channel, list position, 16-bit pattern) for the thread's active channels (only for a
// thread that can own a position in [emit_lo, emit_hi)).  `hint` (top-k; kNoKeyHint = none) is
// a guess of the k-th key that shortens the search and never changes the result; `thr_out`
// (top-k with 0 < k < K) receives the k-th key found, in every thread.  `xchg` (top-k emits; may be NULL) is ceil(K/8) words of shared
// memory apart from the histogram's first KeyWindow bins and from whatever emit writes.
// After a top-k selection with 0 < k < K, s->res[0] holds the k-th
// key until the next selection.
struct NoEmit {
    __device__ __forceinline__ void operator()(int, int, uint16_t) const {}
};

// emit(channel, list position, 16-bit pattern) for the set bits of chunk c's flag byte (w = the
// chunk's four words); the first set bit gets position `pos`.  Eight independent predicated
// calls, no loop over the set bits: nothing waits for the previous channel.
template <class Emit>
__device__ __forceinline__ void emit_chunk(uint32_t byte, int c, const uint32_t (&w)[4], int pos, Emit& emit) {
#pragma unroll
    for (int e = 0; e < 8; ++e)
        if (byte & (1u << e))
            emit((c << 3) + e, pos + __popc(byte & ((1u << e) - 1u)),
                 static_cast<uint16_t>(w[e >> 1] >> (16 * (e & 1))));
}

template <int DT, int NT, class Emit = NoEmit>
__device__ __forceinline__ unsigned long long block_token_flags(const uint16_t* xs, int K, int mode, int k,
                                                                float tau, uint32_t* hist, bool hist_clean,
                                                                SelectScratch* s, bool single, int& pos0,
                                                                int& cnt, Emit emit = Emit(), int emit_lo = 0,
                                                                int emit_hi = 0x7FFFFFFF,
                                                                uint32_t hint = kNoKeyHint,
                                                                uint32_t* xchg = nullptr,
                                                                uint32_t* thr_out = nullptr) {
    int c_lo, c_hi;
    thread_chunk_range(K, c_lo, c_hi);
    unsigned long long fl = 0ull;
    if (mode == AFX_MODE_THRESHOLD || k >= K || k <= 0) {
        const bool all = mode == AFX_MODE_THRESHOLD ? tau < 0.0f : k > 0;
        const bool none = mode != AFX_MODE_THRESHOLD && k <= 0;
        for (int c = c_lo; c < c_hi; ++c) {
            const uint4 raw = *reinterpret_cast<const uint4*>(xs + (c << 3));
            const uint32_t r[4] = {raw.x, raw.y, raw.z, raw.w};
            uint32_t byte = 0;
#pragma unroll
            for (int e = 0; e < 8; ++e) {
                const uint16_t bits = static_cast<uint16_t>(r[e >> 1] >> (16 * (e & 1)));
                const bool in = (c << 3) + e < K;
                const bool pred = in && !none && (all || fabsf(bits_to_float<DT>(bits)) > tau);
                byte |= static_cast<uint32_t>(pred) << e;
            }
            fl |= static_cast<unsigned long long>(byte) << (8 * (c - c_lo));
        }
        if (single) {
            pos0 = block_prefix(__popcll(fl), s->wtot[1], cnt);
            int pos = pos0;
            if (!std::is_same<Emit, NoEmit>::value && pos0 < emit_hi && pos0 + __popcll(fl) > emit_lo) {
                for (int c = c_lo; c < c_hi; ++c) {
                    const uint32_t byte = static_cast<uint32_t>(fl >> (8 * (c - c_lo))) & 0xFFu;
                    if (byte == 0u) continue;
                    const uint4 raw = *reinterpret_cast<const uint4*>(xs + (c << 3));
                    const uint32_t w[4] = {raw.x, raw.y, raw.z, raw.w};
                    emit_chunk(byte, c, w, pos, emit);
                    pos += __popc(byte);
                }
            }
        }
        return fl;
    }
    if (!hist_clean) {
        __syncthreads();  // a hinted search of the previous token may still be read by slower warps
        block_clear_key_hist<NT>(hist);
        __syncthreads();
    }
    uint32_t thr;
    int need_eq, tot_eq;
    if (!(hint != kNoKeyHint && block_kth_key_near<DT, NT>(xs, K, k, hint, hist, s, thr, need_eq, tot_eq)))
        block_kth_key<NT>(xs, K, k, hist, s, thr, need_eq, tot_eq);
    if (thr_out != nullptr) *thr_out = thr;
    AFX_MARK(8);
    // Channels above the k-th key are in; of those equal to it, the need_eq lowest ids.  One
    // pass over the thread's chunks, two keys per operation (swar_*), leaves two flag sets in
    // registers: keys greater than the k-th and keys equal to it.  A partial last chunk is
    // padded with zeros in shared memory; a zero key is never greater, and counts as equal
    // only when thr == 0, so the padding is masked out of the equal flags.
    const uint32_t thr2 = swar_pair(thr), thr2p1 = swar_pair(thr + 1u);
    unsigned long long fg = 0ull, fe = 0ull;
    for (int c = c_lo; c < c_hi; ++c) {
        const uint4 raw = *reinterpret_cast<const uint4*>(xs + (c << 3));
        const uint32_t r[4] = {raw.x & 0x7FFF7FFFu, raw.y & 0x7FFF7FFFu, raw.z & 0x7FFF7FFFu, raw.w & 0x7FFF7FFFu};
        uint32_t gt = 0, ge = 0;  // word i: low key -> bit 2i, high key -> bit 16 + 2i
#pragma unroll
        for (int i = 0; i < 4; ++i) {
            gt |= (swar_gt(r[i], thr2p1) >> (15 - 2 * i)) & (0x00010001u << (2 * i));
            ge |= (swar_gt(r[i], thr2) >> (15 - 2 * i)) & (0x00010001u << (2 * i));  // key > thr - 1
        }
        const uint32_t gbyte = (gt | (gt >> 15)) & 0xFFu;
        uint32_t ebyte = (ge | (ge >> 15)) & 0xFFu & ~gbyte;
        const int nvalid = K - (c << 3);
        if (nvalid < 8) ebyte &= (1u << nvalid) - 1u;
        fg |= static_cast<unsigned long long>(gbyte) << (8 * (c - c_lo));
        fe |= static_cast<unsigned long long>(ebyte) << (8 * (c - c_lo));
    }
    const int g = __popcll(fg), e_cnt = __popcll(fe);
    AFX_MARK(9);
    int pre_e = 0;
    if (single) {
        int tot;
        const int pre = block_prefix((g << 16) | e_cnt, s->wtot[1], tot);  // g < 2^15, e <= 2^15: no carry
        pre_e = pre & 0xFFFF;
        pos0 = (pre >> 16) + min(pre_e, need_eq);
        cnt = k;
    } else if (need_eq != tot_eq) {
        int tot;
        pre_e = block_prefix(e_cnt, s->wtot[1], tot);
    }
    AFX_MARK(10);
    fl = fg;
    if (need_eq == tot_eq) {
        fl |= fe;
    } else {
        // ties across the boundary: the equal channels are kept in channel order until
        // need_eq of them (over the whole vector) are in
        int seen_e = pre_e;
        for (unsigned long long rest = fe; rest != 0ull && seen_e < need_eq; ++seen_e) {
            const unsigned long long low = rest & (0ull - rest);
            rest ^= low;
            fl |= low;
        }
    }
    if (single && !std::is_same<Emit, NoEmit>::value) {
        const int nchunks = (K + 7) >> 3;
        if (xchg != nullptr && nchunks > NT) {
            // Several chunks per thread: the few owners of the positions [emit_lo, emit_hi)
            // would emit chunk after chunk.  Every owner posts (position, flags) of its chunks
            // instead, and the chunks that touch the range are emitted by one thread each.
            int pos = pos0;
            for (int c = c_lo; c < c_hi; ++c) {
                const uint32_t byte = static_cast<uint32_t>(fl >> (8 * (c - c_lo))) & 0xFFu;
                xchg[c] = (static_cast<uint32_t>(pos) << 8) | byte;
                pos += __popc(byte);
            }
            __syncthreads();
            for (int c = threadIdx.x; c < nchunks; c += NT) {
                const uint32_t v = xchg[c];
                const uint32_t byte = v & 0xFFu;
                const int p = static_cast<int>(v >> 8);
                if (byte != 0u && p < emit_hi && p + __popc(byte) > emit_lo) {
                    const uint4 raw = *reinterpret_cast<const uint4*>(xs + (c << 3));
                    const uint32_t w[4] = {raw.x, raw.y, raw.z, raw.w};
                    emit_chunk(byte, c, w, p, emit);
                }
            }
        } else {
            const int n = __popcll(fl);
            if (pos0 < emit_hi && pos0 + n > emit_lo) {
                int pos = pos0;
                for (int c = c_lo; c < c_hi; ++c) {
                    const uint32_t byte = static_cast<uint32_t>(fl >> (8 * (c - c_lo))) & 0xFFu;
                    if (byte == 0u) continue;
                    const uint4 raw = *reinterpret_cast<const uint4*>(xs + (c << 3));
                    const uint32_t w[4] = {raw.x, raw.y, raw.z, raw.w};
                    emit_chunk(byte, c, w, pos, emit);
                    pos += __popc(byte);
                }
            }
        }
    }
    return fl;
}

// Writes the calling thread's flag bytes into a ceil(K/32)-word bitmap in shared memory
// (bit j % 32 of word j / 32) and clears the bytes past the last chunk.  No barrier.
__device__ __forceinline__ void store_flag_bytes(unsigned long long fl, int K, uint32_t* flags) {
    int c_lo, c_hi;
    thread_chunk_range(K, c_lo, c_hi);
    uint8_t* bytes = reinterpret_cast<uint8_t*>(flags);
    for (int c = c_lo; c < c_hi; ++c) bytes[c] = static_cast<uint8_t>(fl >> (8 * (c - c_lo)));
    const int nchunks = (K + 7) >> 3, nbytes = ((K + 31) >> 5) << 2;
    for (int c = nchunks + threadIdx.x; c < nbytes; c += blockDim.x) bytes[c] = 0;
}

// Calls f(j, pos) for every active channel j of the calling thread, ascending, pos = its
// position in the list.
template <class F>
__device__ __forceinline__ void for_each_owned_active(unsigned long long fl, int K, int pos0, F f) {
    int c_lo, c_hi;
    thread_chunk_range(K, c_lo, c_hi);
    int pos = pos0;
    for (int c = c_lo; c < c_hi; ++c) {
        const uint32_t byte = static_cast<uint32_t>(fl >> (8 * (c - c_lo))) & 0xFFu;
#pragma unroll
        for (int e = 0; e < 8; ++e)
            if (byte & (1u << e)) f((c << 3) + e, pos + __popc(byte & ((1u << e) - 1u)));
        pos += __popc(byte);
    }
}

// Copies one token's K 16-bit patterns from global memory into shared memory and zero-fills
// up to the next multiple of 8 elements.  Ends with a block barrier.
__device__ __forceinline__ void block_stage_token(const uint16_t* __restrict__ x, int K, uint16_t* xs) {
    const int Kp = (K + 7) & ~7;
    if ((reinterpret_cast<uintptr_t>(x) & 15u) == 0) {
        const int nfull = K >> 3;
        for (int c = threadIdx.x; c < nfull; c += blockDim.x)
            reinterpret_cast<uint4*>(xs)[c] = reinterpret_cast<const uint4*>(x)[c];
        for (int j = (nfull << 3) + threadIdx.x; j < Kp; j += blockDim.x) xs[j] = j < K ? x[j] : uint16_t(0);
    } else {
        for (int j = threadIdx.x; j < Kp; j += blockDim.x) xs[j] = j < K ? x[j] : uint16_t(0);
    }
    __syncthreads();
}

// ---- large-K path (K > kSelectFastMaxK): keys read from global memory ----

// Warp 0 only.  hist has nbins (multiple of 32, <= 256) counters; walking bins from the
// highest down, finds the bin that holds the k-th element (k is 1-based and must not
// exceed the histogram's total).  res[0] = that bin, res[1] = number of elements in higher
// bins.
__device__ __forceinline__ void find_kth_bin(const int* hist, int nbins, int k, int* res) {
    const int per = nbins >> 5;
    const int l = lane_id();
    int local = 0;
    for (int q = 0; q < per; ++q) local += hist[nbins - 1 - (l * per + q)];
    int incl = local;
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) {
        int n = __shfl_up_sync(0xFFFFFFFFu, incl, o);
        if (l >= o) incl += n;
    }
    const int before = incl - local;
    if (before < k && k <= incl) {
        int run = before;
        for (int q = 0; q < per; ++q) {
            const int bin = nbins - 1 - (l * per + q);
            const int h = hist[bin];
            if (k <= run + h) {
                res[0] = bin;
                res[1] = run;
                break;
            }
            run += h;
        }
    }
}

// Large-K path: fills flags[0..ceil(K/32)) (shared memory) with the union over tokens of the
// per-token active sets.  x is [T][K] in global memory; two histogram passes per token.
template <int DT>
__device__ void block_select_flags_large(const uint16_t* __restrict__ x, int K, int T, int mode, int k,
                                   float tau, uint32_t* flags, SelectScratch* s) {
    const int nwords = (K + 31) >> 5;
    const int lane = lane_id();
    const uint32_t lt_mask = (1u << lane) - 1u;
    int w0, w1;
    warp_word_range(nwords, w0, w1);
    for (int w = w0 + lane; w < w1; w += 32) flags[w] = 0u;  // own range only
    __syncwarp();

    for (int t = 0; t < T; ++t) {
        const uint16_t* xt = x + static_cast<size_t>(t) * K;
        if (mode == AFX_MODE_THRESHOLD) {
            for (int w = w0; w < w1; ++w) {
                const int j = (w << 5) + lane;
                bool pred = false;
                if (j < K) pred = (tau < 0.0f) || (fabsf(bits_to_float<DT>(xt[j])) > tau);
                const uint32_t b = __ballot_sync(0xFFFFFFFFu, pred);
                if (lane == 0) flags[w] |= b;
            }
            continue;
        }
        // ---- top-k ----
        if (k <= 0) continue;
        if (k >= K) {
            for (int w = w0; w < w1; ++w) {
                const uint32_t b = __ballot_sync(0xFFFFFFFFu, (w << 5) + lane < K);
                if (lane == 0) flags[w] |= b;
            }
            continue;
        }
        // pass 1: histogram of the 8 high key bits
        __syncthreads();
        for (int i = threadIdx.x; i < 256; i += blockDim.x) s->hist[i] = 0;
        __syncthreads();
        for (int j = threadIdx.x; j < K; j += blockDim.x) atomicAdd(&s->hist[mag_key(xt[j]) >> 7], 1);
        __syncthreads();
        if (warp_id() == 0) find_kth_bin(s->hist, 256, k, s->res);
        __syncthreads();
        const uint32_t hi = static_cast<uint32_t>(s->res[0]);
        const int k2 = k - s->res[1];  // rank of the k-th element inside its high-bits bin
        // pass 2: histogram of the 7 low key bits inside that bin
        for (int i = threadIdx.x; i < 128; i += blockDim.x) s->hist[i] = 0;
        __syncthreads();
        for (int j = threadIdx.x; j < K; j += blockDim.x) {
            const uint32_t key = mag_key(xt[j]);
            if ((key >> 7) == hi) atomicAdd(&s->hist[key & 127u], 1);
        }
        __syncthreads();
        if (warp_id() == 0) find_kth_bin(s->hist, 128, k2, s->res + 2);
        __syncthreads();
        const uint32_t thr = (hi << 7) | static_cast<uint32_t>(s->res[2]);  // the k-th largest key
        const int need_eq = k2 - s->res[3];  // how many channels with key == thr are kept
        const bool all_eq = (need_eq == s->hist[s->res[2]]);
        if (all_eq) {
            for (int w = w0; w < w1; ++w) {
                const int j = (w << 5) + lane;
                const bool pred = j < K && mag_key(xt[j]) >= thr;
                const uint32_t b = __ballot_sync(0xFFFFFFFFu, pred);
                if (lane == 0) flags[w] |= b;
            }
        } else {
            // ties at the boundary: keep the need_eq lowest channel ids among key == thr
            int ce = 0;
            for (int w = w0; w < w1; ++w) {
                const int j = (w << 5) + lane;
                ce += __popc(__ballot_sync(0xFFFFFFFFu, j < K && mag_key(xt[j]) == thr));
            }
            int base = block_exclusive_over_warps(ce, s->scan);
            for (int w = w0; w < w1; ++w) {
                const int j = (w << 5) + lane;
                const uint32_t key = j < K ? mag_key(xt[j]) : 0u;
                const bool eq = j < K && key == thr;
                const uint32_t e = __ballot_sync(0xFFFFFFFFu, eq);
                const bool pred = j < K && (key > thr || (eq && base + __popc(e & lt_mask) < need_eq));
                const uint32_t b = __ballot_sync(0xFFFFFFFFu, pred);
                if (lane == 0) flags[w] |= b;
                base += __popc(e);
            }
        }
    }
    __syncthreads();
}

}  // namespace afx
