/*
 * afx_oracle.c -- plain CPU oracle for the active-weight hot path of ActiveFlow's
 * decoding step (arXiv 2504.08378).
 *
 * THIS IS TEST INFRASTRUCTURE.  It is a slow, literal restatement of what the path
 * computes, used only by the test-suite, the smoke check and the benchmark's CPU
 * baseline.  It shares no code with the CUDA library and the CUDA library never
 * calls it.  All floating point is carried in fp64; every rounding to a 16-bit
 * storage type is a single round-to-nearest-even from the fp64 value.
 *
 * What each function follows:
 *   afxo_select_active  Sec. 2.1 ("only the activation elements with a magnitude above a
 *                       threshold will be computed"), Sec. 4 operation "T" (Top-K mask ->
 *                       indices of the activated channels), Sec. 6 "Caching" (the kernel that
 *                       generates active channel indices from per-sparsity thresholds).
 *   afxo_diff_active    Sec. 3 / Fig. "Cross-layer active weight pre-loading": channels the
 *                       prediction missed are the ones fetched on demand.
 *   afxo_sparse_gemv    Sec. 2.1: the operator is evaluated on the active channels only.
 *   afxo_cache_step     Sec. 4.2 "Dynamic LLM Weight Caching" and its worked example.
 *   afxo_rmsnorm/rope/attention/silu_mul
 *                       the decoder layer of Fig. "simplified transformer layer structure";
 *                       the paper is silent on their arithmetic, they are the textbook
 *                       Llama routines.
 *
 * Parity pins (tests/test_oracle_*.py): hand-worked K=8 cases, brute force by an
 * independent numpy implementation, dense==sparse identities, the paper's cache
 * example, numpy/torch fp64 restatements of the textbook layer routines.
 *
 * Storage types: dtype 0 = IEEE binary16 (fp16), dtype 1 = bfloat16; both are passed as
 * uint16_t bit patterns.  Weights are channel-contiguous: input channel j of an operator
 * W in R^{N x K} is the run Wt[j*ldw .. j*ldw+N).
 */
#include <math.h>
#include <stdint.h>
#include <stdlib.h>
#include <string.h>
#ifdef _OPENMP
#include <omp.h>
#endif

#define AFXO_F16 0
#define AFXO_BF16 1
#define AFXO_TOPK 0
#define AFXO_THRESHOLD 1

/* ---------------------------------------------------------------- 16-bit formats */

/* value of a binary16 bit pattern, from the definition of the format */
static double f16_value(uint16_t h)
{
    int sign = (h >> 15) & 1;
    int e = (h >> 10) & 0x1F;
    int m = h & 0x3FF;
    double v;
    if (e == 0)
        v = ldexp((double)m, -24); /* subnormal: m * 2^-10 * 2^-14 */
    else if (e == 31)
        v = m ? NAN : INFINITY;
    else
        v = ldexp(1.0 + (double)m / 1024.0, e - 15);
    return sign ? -v : v;
}

/* value of a bfloat16 bit pattern: sign, 8 exponent bits (bias 127), 7 fraction bits */
static double bf16_value(uint16_t b)
{
    int sign = (b >> 15) & 1;
    int e = (b >> 7) & 0xFF;
    int m = b & 0x7F;
    double v;
    if (e == 0)
        v = ldexp((double)m, -133); /* m * 2^-7 * 2^-126 */
    else if (e == 255)
        v = m ? NAN : INFINITY;
    else
        v = ldexp(1.0 + (double)m / 128.0, e - 127);
    return sign ? -v : v;
}

static double value_of(uint16_t bits, int dtype)
{
    return dtype == AFXO_F16 ? f16_value(bits) : bf16_value(bits);
}

/* Round an fp64 value once, to nearest-even, into a format with `p` significant bits,
 * minimum normal exponent emin and maximum exponent emax, and return its bit pattern in
 * a layout of (1 sign, ebits exponent, p-1 fraction). */
static uint16_t round_to_bits(double v, int p, int ebits)
{
    int bias = (1 << (ebits - 1)) - 1;
    int emin = 1 - bias, emax = bias;
    uint16_t sign = signbit(v) ? (uint16_t)0x8000 : 0;
    uint16_t expo_all = (uint16_t)(((1 << ebits) - 1) << (p - 1));
    if (isnan(v))
        return (uint16_t)(sign | expo_all | (1 << (p - 2)));
    double a = fabs(v);
    if (isinf(a))
        return (uint16_t)(sign | expo_all);
    if (a == 0.0)
        return sign;
    int e;
    frexp(a, &e); /* a = f * 2^e with 0.5 <= f < 1: leading bit has weight 2^(e-1) */
    int lead = e - 1;
    if (lead < emin)
        lead = emin;
    double ulp = ldexp(1.0, lead - (p - 1));
    double q = rint(a / ulp); /* scaling by a power of two is exact; rint is ties-to-even */
    double r = q * ulp;
    if (r >= ldexp(1.0, emax + 1))
        return (uint16_t)(sign | expo_all); /* overflow rounds to infinity */
    if (r == 0.0)
        return sign;
    frexp(r, &e);
    lead = e - 1;
    if (lead < emin) { /* subnormal: exponent field 0, fraction = r / 2^(emin-(p-1)) */
        uint16_t frac = (uint16_t)(r / ldexp(1.0, emin - (p - 1)));
        return (uint16_t)(sign | frac);
    }
    double frac_d = (r / ldexp(1.0, lead) - 1.0) * (double)(1 << (p - 1));
    return (uint16_t)(sign | ((uint16_t)(lead + bias) << (p - 1)) | (uint16_t)frac_d);
}

static uint16_t round_dtype(double v, int dtype)
{
    return dtype == AFXO_F16 ? round_to_bits(v, 11, 5) : round_to_bits(v, 8, 8);
}

/* exported for the tests that pin the format code against numpy / torch */
void afxo_decode(const uint16_t* bits, int64_t n, int dtype, double* out)
{
    for (int64_t i = 0; i < n; ++i)
        out[i] = value_of(bits[i], dtype);
}

void afxo_round(const double* v, int64_t n, int dtype, uint16_t* out)
{
    for (int64_t i = 0; i < n; ++i)
        out[i] = round_dtype(v[i], dtype);
}

/* ---------------------------------------------------------------- selection */

typedef struct {
    uint16_t key; /* |x| as an integer: the bit pattern with the sign cleared */
    int32_t j;
} afxo_keyed;

/* larger magnitude first; among equal magnitudes the lower channel index first */
static int keyed_before(const void* pa, const void* pb)
{
    const afxo_keyed* a = (const afxo_keyed*)pa;
    const afxo_keyed* b = (const afxo_keyed*)pb;
    if (a->key != b->key)
        return a->key > b->key ? -1 : 1;
    return a->j < b->j ? -1 : (a->j > b->j ? 1 : 0);
}

/*
 * Active channels of T activation vectors x[t][0..K).
 *   mode TOPK:      per token, the k channels of largest |x|, ties to the lower index
 *                   (literal full sort).  For finite values the sign-cleared bit pattern
 *                   orders exactly like |x|; a NaN pattern ranks above infinity.
 *   mode THRESHOLD: per token, channels with (float)|x_j| > tau ("above", strict); a NaN
 *                   never compares above.  tau < 0 keeps every channel.
 * The result for T > 1 is the union over tokens.  idx receives the active channel ids in
 * ascending order, *count their number.  Returns 0, or -1 on a bad argument.
 */
int afxo_select_active(const uint16_t* x, int dtype, int K, int T, int mode, int k, float tau,
                       int32_t* idx, int32_t* count)
{
    if (!x || !idx || !count || K <= 0 || T <= 0 || (dtype != AFXO_F16 && dtype != AFXO_BF16))
        return -1;
    if (mode == AFXO_TOPK && (k < 0 || k > K))
        return -1;
    if (mode != AFXO_TOPK && mode != AFXO_THRESHOLD)
        return -1;
    unsigned char* active = (unsigned char*)calloc((size_t)K, 1);
    afxo_keyed* order = (afxo_keyed*)malloc(sizeof(afxo_keyed) * (size_t)K);
    for (int t = 0; t < T; ++t) {
        const uint16_t* xt = x + (size_t)t * K;
        if (mode == AFXO_TOPK) {
            for (int j = 0; j < K; ++j) {
                order[j].key = (uint16_t)(xt[j] & 0x7FFF);
                order[j].j = j;
            }
            qsort(order, (size_t)K, sizeof(afxo_keyed), keyed_before);
            for (int r = 0; r < k; ++r)
                active[order[r].j] = 1;
        } else {
            for (int j = 0; j < K; ++j) {
                if (tau < 0.0f) {
                    active[j] = 1;
                } else {
                    float mag = (float)fabs(value_of(xt[j], dtype)); /* exact: 16-bit -> fp32 */
                    if (mag > tau)
                        active[j] = 1;
                }
            }
        }
    }
    int32_t n = 0;
    for (int j = 0; j < K; ++j)
        if (active[j])
            idx[n++] = j;
    *count = n;
    free(order);
    free(active);
    return 0;
}

/*
 * Cross-layer bookkeeping: A = actual active set of a layer, P = the set predicted for it
 * by an earlier layer (both ascending).  miss = A \ P ascending (the channels fetched on
 * demand), *hit_count = |A intersect P|.
 */
int afxo_diff_active(const int32_t* idxA, int32_t cntA, const int32_t* idxP, int32_t cntP, int K,
                     int32_t* miss, int32_t* miss_count, int32_t* hit_count)
{
    if (K <= 0 || cntA < 0 || cntP < 0)
        return -1;
    unsigned char* inP = (unsigned char*)calloc((size_t)K, 1);
    for (int32_t c = 0; c < cntP; ++c)
        inP[idxP[c]] = 1;
    int32_t nm = 0, nh = 0;
    for (int32_t c = 0; c < cntA; ++c) {
        if (inP[idxA[c]])
            ++nh;
        else
            miss[nm++] = idxA[c];
    }
    *miss_count = nm;
    *hit_count = nh;
    free(inP);
    return 0;
}

/* ---------------------------------------------------------------- sparse GEMV */

/*
 * y[t][i] = sum over c in [0,cnt), ascending, of x[t][idx[c]] * Wt[col(c)*ldw + i], all in
 * fp64.  col(c) = idx[c], or slot[c] when a slot list is given (columns living in a cache).
 * Output rows are independent, so the loop over i may be shared between threads without
 * changing any sum's order.
 */
int afxo_sparse_gemv(const uint16_t* Wt, int dtype, int K, int N, int64_t ldw, const uint16_t* x,
                     int T, const int32_t* idx, int32_t cnt, const int32_t* slot, double* y)
{
    if (!Wt || !x || !y || K <= 0 || N <= 0 || T <= 0 || ldw < N || cnt < 0 || cnt > K)
        return -1;
    for (int t = 0; t < T; ++t) {
        double* yt = y + (size_t)t * N;
        const uint16_t* xt = x + (size_t)t * K;
#pragma omp parallel for schedule(static)
        for (int ib = 0; ib < N; ib += 256) {
            int ie = ib + 256 < N ? ib + 256 : N;
            for (int i = ib; i < ie; ++i)
                yt[i] = 0.0;
            for (int32_t c = 0; c < cnt; ++c) {
                int32_t j = idx[c];
                const uint16_t* col = Wt + (size_t)(slot ? slot[c] : j) * (size_t)ldw;
                double xj = value_of(xt[j], dtype);
                for (int i = ib; i < ie; ++i)
                    yt[i] += xj * value_of(col[i], dtype);
            }
        }
    }
    return 0;
}

int afxo_threads(void)
{
#ifdef _OPENMP
    return omp_get_max_threads();
#else
    return 1;
#endif
}

/* Caps the threads the row-parallel loops may use (timing the oracle on one core); no effect
 * on any result: every output row is summed by one thread in the same order. */
void afxo_set_threads(int n)
{
#ifdef _OPENMP
    if (n >= 1)
        omp_set_num_threads(n);
#else
    (void)n;
#endif
}

/* ---------------------------------------------------------------- decoder-layer glue */

/* out[t][j] = round_dtype( h[t][j] / sqrt(mean_j h^2 + eps) * g[j] ) */
void afxo_rmsnorm(const double* h, const double* g, int T, int H, double eps, int dtype,
                  uint16_t* out)
{
    for (int t = 0; t < T; ++t) {
        const double* ht = h + (size_t)t * H;
        double ss = 0.0;
        for (int j = 0; j < H; ++j)
            ss += ht[j] * ht[j];
        double inv = 1.0 / sqrt(ss / (double)H + eps);
        for (int j = 0; j < H; ++j)
            out[(size_t)t * H + j] = round_dtype(ht[j] * inv * g[j], dtype);
    }
}

/*
 * Rotary embedding on adjacent pairs (v[2i], v[2i+1]) of every head of v[t][head][D]:
 * angle = pos[t] * theta^(-2i/D).  In place.
 */
void afxo_rope(double* v, int T, int heads, int D, const int32_t* pos, double theta)
{
    for (int t = 0; t < T; ++t)
        for (int hd = 0; hd < heads; ++hd) {
            double* p = v + ((size_t)t * heads + hd) * D;
            for (int i = 0; i < D / 2; ++i) {
                double ang = (double)pos[t] * pow(theta, -2.0 * (double)i / (double)D);
                double c = cos(ang), s = sin(ang);
                double a = p[2 * i], b = p[2 * i + 1];
                p[2 * i] = a * c - b * s;
                p[2 * i + 1] = a * s + b * c;
            }
        }
}

/*
 * Dense single-query attention for one token over a key/value cache held in fp16 bits:
 * kc, vc are [L][kv_heads][D] with L valid positions (the current token's k, v already
 * appended by the caller).  q is [q_heads][D] fp64; query head hq reads kv head
 * hq / (q_heads / kv_heads).  out[hq][:] = softmax(q.k / sqrt(D)) . v, then rounded to
 * dtype bits.
 */
void afxo_attention(const double* q, const uint16_t* kc, const uint16_t* vc, int L, int q_heads,
                    int kv_heads, int D, int dtype, uint16_t* out)
{
    int rep = q_heads / kv_heads;
    double scale = 1.0 / sqrt((double)D);
    double* s = (double*)malloc(sizeof(double) * (size_t)L);
    double* acc = (double*)malloc(sizeof(double) * (size_t)D);
    for (int hq = 0; hq < q_heads; ++hq) {
        int hk = hq / rep;
        const double* qh = q + (size_t)hq * D;
        double mx = -INFINITY;
        for (int l = 0; l < L; ++l) {
            const uint16_t* kl = kc + ((size_t)l * kv_heads + hk) * D;
            double d = 0.0;
            for (int i = 0; i < D; ++i)
                d += qh[i] * f16_value(kl[i]);
            s[l] = d * scale;
            if (s[l] > mx)
                mx = s[l];
        }
        double z = 0.0;
        for (int l = 0; l < L; ++l) {
            s[l] = exp(s[l] - mx);
            z += s[l];
        }
        for (int i = 0; i < D; ++i)
            acc[i] = 0.0;
        for (int l = 0; l < L; ++l) {
            const uint16_t* vl = vc + ((size_t)l * kv_heads + hk) * D;
            double p = s[l] / z;
            for (int i = 0; i < D; ++i)
                acc[i] += p * f16_value(vl[i]);
        }
        for (int i = 0; i < D; ++i)
            out[(size_t)hq * D + i] = round_dtype(acc[i], dtype);
    }
    free(acc);
    free(s);
}

/* out[i] = round_dtype( g[i] / (1 + exp(-g[i])) * u[i] ) */
void afxo_silu_mul(const double* g, const double* u, int64_t n, int dtype, uint16_t* out)
{
    for (int64_t i = 0; i < n; ++i)
        out[i] = round_dtype(g[i] / (1.0 + exp(-g[i])) * u[i], dtype);
}

/* ---------------------------------------------------------------- weight cache */

/*
 * One decoding step of the context-level least-frequently-used column cache of one weight
 * tensor (Sec. 4.2).  State: slot_of[K] (slot holding channel j, or -1), chan_of[C] (channel
 * in slot s, or -1 when free), freq[K] (times channel j was active in this sequence; the
 * caller zeroes it at sequence start).
 *
 * For the ascending active list idx[0..cnt):
 *   1. freq[j] += 1 for every active j.
 *   2. A channel already in a slot is a hit.
 *   3. Misses are handled in ascending channel order.  With a free slot: take the lowest
 *      free slot.  Otherwise the victim is the cached channel that is not active in this
 *      step with the smallest (freq, channel id); the miss replaces it when
 *      freq[miss] >= freq[victim] (the worked example replaces on equal counts).  A miss
 *      that cannot replace anything is "transient": used for this step from a staging slot,
 *      not kept.
 * slot_out[c] = slot of idx[c] after the step; transient misses get C + (their rank among
 * this step's transients).  fetched[0..*n_fetch) lists the missed channels in order.
 */
int afxo_cache_step(int K, int C, int32_t* slot_of, int32_t* chan_of, uint32_t* freq,
                    const int32_t* idx, int32_t cnt, int32_t* slot_out, int32_t* fetched,
                    int32_t* n_hit, int32_t* n_miss, int32_t* n_transient)
{
    if (K <= 0 || C <= 0 || C > K || cnt < 0 || cnt > K)
        return -1;
    unsigned char* active = (unsigned char*)calloc((size_t)K, 1);
    for (int32_t c = 0; c < cnt; ++c) {
        active[idx[c]] = 1;
        freq[idx[c]] += 1;
    }
    int32_t hits = 0, misses = 0, transients = 0;
    for (int32_t c = 0; c < cnt; ++c) {
        int32_t j = idx[c];
        if (slot_of[j] >= 0) {
            ++hits;
            slot_out[c] = slot_of[j];
            continue;
        }
        fetched[misses++] = j;
        int32_t s = -1;
        for (int32_t f = 0; f < C; ++f)
            if (chan_of[f] < 0) {
                s = f;
                break;
            }
        if (s < 0) {
            int32_t victim = -1;
            for (int32_t f = 0; f < C; ++f) {
                int32_t v = chan_of[f];
                if (active[v])
                    continue;
                if (victim < 0 || freq[v] < freq[victim] || (freq[v] == freq[victim] && v < victim))
                    victim = v;
            }
            if (victim >= 0 && freq[j] >= freq[victim]) {
                s = slot_of[victim];
                slot_of[victim] = -1;
            }
        }
        if (s >= 0) {
            chan_of[s] = j;
            slot_of[j] = s;
            slot_out[c] = s;
        } else {
            slot_out[c] = C + transients;
            ++transients;
        }
    }
    *n_hit = hits;
    *n_miss = misses;
    *n_transient = transients;
    free(active);
    return 0;
}
