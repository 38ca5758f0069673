// afx_model_* / afx_state_* / afx_layer_step / afx_mlp_block: a decoder layer as five kernels.
#include <math.h>
#include <new>
#include <vector>

#include "afx_attn.cuh"
#include "afx_fused.cuh"
#include "afx_launch.cuh"
#include "afx_q4.cuh"

namespace afx {

template <int TMAX>
struct FusedShape {
    static constexpr int kBlocksPerSM = TMAX <= 1 ? 2 : 1;
    static constexpr int kStageCap = TMAX <= 4 ? 2048 : 1024;
};

template <int DT, int TMAX, int PW, int IN, int EP>
__global__ void __launch_bounds__(kGemvThreads, FusedShape<TMAX>::kBlocksPerSM)
fused_op_kernel(FusedArgs a) {
    constexpr int CAP = FusedShape<TMAX>::kStageCap;
    extern __shared__ __align__(16) unsigned char dyn[];
    __shared__ SelectScratch sel;
    __shared__ GemvRecv<TMAX> recv;
    fused_op_block<DT, TMAX, PW, CAP, IN, EP>(a, dyn, &sel, &recv);
}

// The operator for several tokens per step: the streaming stage runs on the tensor cores.  The
// block is alone on its SM: staged entries per pass as many as the inputs of TMAX tokens leave room for.
constexpr int kFusedMtStages = 3, kFusedMtStagesSmall = 2;  // pipeline stages of the several-token operator
constexpr size_t kMaxDynSmem = 227 * 1024;
template <int TMAX>
struct FusedMtCap {
    static constexpr int value = TMAX <= 4 ? 4096 : 1024;  // (multiples of kFusedMtRows)
};
// CAPM staged entries per pass, STAGES pipeline stages, BPS blocks per SM.
template <int DT, int TMAX, int IN, int EP, int STAGES, int CAPM, int BPS>
__global__ void __launch_bounds__(kGemvThreads, BPS) fused_mt_kernel(FusedArgs a) {
    extern __shared__ __align__(16) unsigned char dyn[];
    __shared__ SelectScratch sel;
    fused_op_block<DT, TMAX, kMtTile, CAPM, IN, EP, false, false, STAGES>(a, dyn, &sel, nullptr);
}

// The one-token operator for a family of `groups` operators in one grid (mixture of experts).
template <int DT, int PW, int IN, int EP>
__global__ void __launch_bounds__(kGemvThreads, 2) fused_family_kernel(FusedArgs a) {
    constexpr int CAP = FusedShape<1>::kStageCap;
    extern __shared__ __align__(16) unsigned char dyn[];
    __shared__ SelectScratch sel;
    __shared__ GemvRecv<1> recv;
    fused_op_block<DT, 1, PW, CAP, IN, EP, false, true>(a, dyn, &sel, &recv);
}

// The one-token operator over 4-bit rows: tiles of PW = 512, 256 or 128 outputs.
template <int DT, int PW, int IN, int EP>
__global__ void __launch_bounds__(kGemvThreads, 2) fused_q4_kernel(FusedArgs a) {
    constexpr int CAP = FusedShape<1>::kStageCap;
    extern __shared__ __align__(16) unsigned char dyn[];
    __shared__ SelectScratch sel;
    fused_op_block<DT, 1, PW, CAP, IN, EP, true>(a, dyn, &sel, nullptr);
}

template <int DT, int REP>
__global__ void __launch_bounds__(kAttnThreads, REP <= 2 ? 2 : 1) attention_kernel(AttnArgs a) {
    __shared__ AttnSmem sm;
    attention_block<DT, REP>(a, &sm);
}

template <int DT>
static cudaError_t launch_attention_rep(const cudaLaunchConfig_t& cfg, int rep, const AttnArgs& a) {
    if (rep <= 1) return cudaLaunchKernelEx(&cfg, attention_kernel<DT, 1>, a);
    if (rep <= 2) return cudaLaunchKernelEx(&cfg, attention_kernel<DT, 2>, a);
    if (rep <= 4) return cudaLaunchKernelEx(&cfg, attention_kernel<DT, 4>, a);
    return cudaLaunchKernelEx(&cfg, attention_kernel<DT, 8>, a);
}

template <int DT, int TMAX, int IN, int EP>
static afx_status launch_fused_t(const FusedArgs& a, cudaStream_t st) {
    // staged column offsets are 32-bit counts of 16-byte units
    if (static_cast<uint64_t>(a.K) * static_cast<uint64_t>(a.ldw >> 3) > 0x100000000ull) return AFX_ERR_CAPACITY;
    const size_t dyn = fused_dyn_smem(IN, a.K, a.T);
    const void* kerns[3] = {reinterpret_cast<const void*>(fused_op_kernel<DT, TMAX, 256, IN, EP>),
                            reinterpret_cast<const void*>(fused_op_kernel<DT, TMAX, 128, IN, EP>),
                            reinterpret_cast<const void*>(fused_op_kernel<DT, TMAX, 64, IN, EP>)};
    // side outputs, if any, come from one more cluster than there are column tiles
    FusedArgs b = a;
    b.side_cluster = (a.idx_out != nullptr || a.count_out != nullptr || a.bitmap_out != nullptr ||
                      a.xnorm_out != nullptr || a.bitmap_pred != nullptr || a.kth_slot != nullptr ||
                      (a.kth_multi != nullptr && a.T > 1))
                         ? 1 : 0;
    const GemvShapeChoice c = choose_gemv_shape(a.N, kerns, dyn, b.side_cluster);
    if (c.tiles + b.side_cluster > 65535) return AFX_ERR_CAPACITY;
    const int rows = c.tiles + b.side_cluster;
    switch (c.pw) {
        case 256: return launch_clustered(fused_op_kernel<DT, TMAX, 256, IN, EP>, c.S, rows, dyn, b, st);
        case 128: return launch_clustered(fused_op_kernel<DT, TMAX, 128, IN, EP>, c.S, rows, dyn, b, st);
        default: return launch_clustered(fused_op_kernel<DT, TMAX, 64, IN, EP>, c.S, rows, dyn, b, st);
    }
}

// `groups` operators of one family (weights from a.wt_table through a.wt_sel[g]) in one grid;
// one token, no side outputs.
template <int DT, int IN, int EP>
static afx_status launch_fused_family_dt(const FusedArgs& a, cudaStream_t st) {
    if (static_cast<uint64_t>(a.K) * static_cast<uint64_t>(a.ldw >> 3) > 0x100000000ull) return AFX_ERR_CAPACITY;
    if (a.T != 1 || a.groups < 1 || a.wt_table == nullptr || a.wt_sel == nullptr) return AFX_ERR_INVALID_ARG;
    const size_t dyn = fused_dyn_smem(IN, a.K, 1);
    const void* kerns[3] = {reinterpret_cast<const void*>(fused_family_kernel<DT, 256, IN, EP>),
                            reinterpret_cast<const void*>(fused_family_kernel<DT, 128, IN, EP>),
                            reinterpret_cast<const void*>(fused_family_kernel<DT, 64, IN, EP>)};
    FusedArgs b = a;
    b.side_cluster = 0;
    const GemvShapeChoice c = choose_gemv_shape(a.N, kerns, dyn, 0, 256, a.groups);
    if (c.tiles > 65535) return AFX_ERR_CAPACITY;
    switch (c.pw) {
        case 256: return launch_clustered(fused_family_kernel<DT, 256, IN, EP>, c.S, c.tiles, dyn, b, st);
        case 128: return launch_clustered(fused_family_kernel<DT, 128, IN, EP>, c.S, c.tiles, dyn, b, st);
        default: return launch_clustered(fused_family_kernel<DT, 64, IN, EP>, c.S, c.tiles, dyn, b, st);
    }
}

template <int IN, int EP>
static afx_status launch_fused_family(int dtype, const FusedArgs& a, cudaStream_t st) {
    return dtype == AFX_F16 ? launch_fused_family_dt<AFX_F16, IN, EP>(a, st) : launch_fused_family_dt<AFX_BF16, IN, EP>(a, st);
}

// a.Wt = the 4-bit rows, a.ldw = their stride in units of 2 bytes, a.T == 1, a.N % 32 == 0.
template <int DT, int IN, int EP>
static afx_status launch_fused_q4_dt(const FusedArgs& a, cudaStream_t st) {
    if (static_cast<uint64_t>(a.K) * static_cast<uint64_t>(a.ldw >> 3) > 0x100000000ull) return AFX_ERR_CAPACITY;
    const size_t dyn = fused_dyn_smem(IN, a.K, 1);
    const void* kerns[3] = {reinterpret_cast<const void*>(fused_q4_kernel<DT, 512, IN, EP>),
                            reinterpret_cast<const void*>(fused_q4_kernel<DT, 256, IN, EP>),
                            reinterpret_cast<const void*>(fused_q4_kernel<DT, 128, IN, EP>)};
    FusedArgs b = a;
    b.side_cluster = (a.idx_out != nullptr || a.count_out != nullptr || a.bitmap_out != nullptr ||
                      a.xnorm_out != nullptr || a.bitmap_pred != nullptr || a.kth_slot != nullptr)
                         ? 1 : 0;
    const GemvShapeChoice c = choose_gemv_shape(a.N, kerns, dyn, b.side_cluster, 512);
    if (c.tiles + b.side_cluster > 65535) return AFX_ERR_CAPACITY;
    const int rows = c.tiles + b.side_cluster;
    switch (c.pw) {
        case 512: return launch_clustered(fused_q4_kernel<DT, 512, IN, EP>, c.S, rows, dyn, b, st);
        case 256: return launch_clustered(fused_q4_kernel<DT, 256, IN, EP>, c.S, rows, dyn, b, st);
        default: return launch_clustered(fused_q4_kernel<DT, 128, IN, EP>, c.S, rows, dyn, b, st);
    }
}

template <int IN, int EP>
static afx_status launch_fused_q4(int dtype, const FusedArgs& a, cudaStream_t st) {
    return dtype == AFX_F16 ? launch_fused_q4_dt<AFX_F16, IN, EP>(a, st) : launch_fused_q4_dt<AFX_BF16, IN, EP>(a, st);
}


template <int DT, int TMAX, int IN, int EP, int STAGES, int CAPM, int BPS>
static afx_status launch_fused_mt_st(const FusedArgs& a, cudaStream_t st) {
    const void* kern = reinterpret_cast<const void*>(fused_mt_kernel<DT, TMAX, IN, EP, STAGES, CAPM, BPS>);
    const size_t dyn = fused_dyn_smem(IN, a.K, a.T, sizeof(MtSmem<CAPM, STAGES, kFusedMtRows>));
    FusedArgs b = a;
    b.side_cluster = (a.idx_out != nullptr || a.count_out != nullptr || a.bitmap_out != nullptr ||
                      a.xnorm_out != nullptr || a.bitmap_pred != nullptr || a.kth_slot != nullptr ||
                      a.kth_multi != nullptr)
                         ? 1 : 0;
    const int tiles = (a.N + kMtTile - 1) / kMtTile;
    if (tiles + b.side_cluster > 65535) return AFX_ERR_CAPACITY;
    const int margin = (tiles + 15) / 16 < 2 ? 2 : (tiles + 15) / 16;
    int S = 1;
    for (int s = kMaxCluster; s > 1; --s)
        if (max_active_clusters(kern, s, dyn) >= tiles + b.side_cluster + margin) {
            S = s;
            break;
        }
    // Few tiles leave the clusters smaller than the number of tokens: let a cluster cover several
    // adjacent tiles, so that its blocks share the per-token selections (own selection only).
    int tpc = 1;
    if (a.idx_in == nullptr)
        for (int t2 = 8; t2 > 1; t2 >>= 1) {
            const int cs = S * t2, rows2 = (tiles + t2 - 1) / t2 + b.side_cluster;
            if (cs <= kMaxCluster && cs <= 2 * a.T && max_active_clusters(kern, cs, dyn) >= rows2 + (margin + t2 - 1) / t2) {
                tpc = t2;
                break;
            }
        }
    b.tiles_per_cluster = tpc;
    const int rows = (tiles + tpc - 1) / tpc + b.side_cluster;
    return launch_clustered(fused_mt_kernel<DT, TMAX, IN, EP, STAGES, CAPM, BPS>, S * tpc, rows, dyn, b, st);
}

// One block per SM (the inputs of several tokens and the tensor-core buffers fill its shared
// memory): 3 pipeline stages of 64 channels, 2 where 8 tokens of a wide model leave less.  (Two blocks per SM
// with the buffers inside the histogram's 64 KB -- 512 staged entries per pass, 3 stages, twice
// as many blocks to share the per-token selections -- measured slower: 295 instead of 255 us per
// 13B layer at 4 tokens.)
template <int DT, int TMAX, int IN, int EP>
static afx_status launch_fused_mt(const FusedArgs& a, cudaStream_t st) {
    if (static_cast<uint64_t>(a.K) * static_cast<uint64_t>(a.ldw >> 3) > 0x100000000ull) return AFX_ERR_CAPACITY;
    constexpr int kCap1 = FusedMtCap<TMAX>::value;
    if (fused_dyn_smem(IN, a.K, a.T, sizeof(MtSmem<kCap1, kFusedMtStages, kFusedMtRows>)) <= kMaxDynSmem)
        return launch_fused_mt_st<DT, TMAX, IN, EP, kFusedMtStages, kCap1, 1>(a, st);
    if (fused_dyn_smem(IN, a.K, a.T, sizeof(MtSmem<kCap1, kFusedMtStagesSmall, kFusedMtRows>)) <= kMaxDynSmem)
        return launch_fused_mt_st<DT, TMAX, IN, EP, kFusedMtStagesSmall, kCap1, 1>(a, st);
    return AFX_ERR_CAPACITY;
}

template <int DT, int IN, int EP>
static afx_status launch_fused_dt(const FusedArgs& a, cudaStream_t st) {
    if (a.T <= 1) return launch_fused_t<DT, 1, IN, EP>(a, st);
    if (a.T <= 4) return launch_fused_mt<DT, 4, IN, EP>(a, st);
    return launch_fused_mt<DT, 8, IN, EP>(a, st);
}

template <int IN, int EP>
static afx_status launch_fused(int dtype, const FusedArgs& a, cudaStream_t st) {
    return dtype == AFX_F16 ? launch_fused_dt<AFX_F16, IN, EP>(a, st) : launch_fused_dt<AFX_BF16, IN, EP>(a, st);
}

static afx_status launch_attention(int dtype, const AttnArgs& a, cudaStream_t st) {
    // split the cached positions so that kv_heads * T * S blocks fill the machine, S <= 8
    const int groups = a.kv_heads * a.T;
    int S = (2 * sm_count() + groups - 1) / groups;
    S = S < 1 ? 1 : (S > 8 ? 8 : S);
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3(S, a.kv_heads, a.T);
    cfg.blockDim = dim3(kAttnThreads, 1, 1);
    cfg.stream = st;
    cudaLaunchAttribute attr[2];
    attr[0].id = cudaLaunchAttributeClusterDimension;
    attr[0].val.clusterDim.x = S;
    attr[0].val.clusterDim.y = 1;
    attr[0].val.clusterDim.z = 1;
    attr[1].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[1].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr;
    cfg.numAttrs = 2;
    const int rep = a.q_heads / a.kv_heads;
    const cudaError_t e = dtype == AFX_F16 ? launch_attention_rep<AFX_F16>(cfg, rep, a)
                                           : launch_attention_rep<AFX_BF16>(cfg, rep, a);
    return e == cudaSuccess ? AFX_OK : AFX_ERR_CUDA;
}

static size_t align256(size_t b) { return (b + 255) / 256 * 256; }

}  // namespace afx

struct afx_model {
    afx_model_desc d;
    std::vector<afx_layer_desc> layers;
    float* rope = nullptr;  // DEVICE: cos[max_seq][64] then sin[max_seq][64]
    int n_qkv = 0;
    int K_op[4] = {0, 0, 0, 0};
};

struct afx_state {
    const afx_model* model;
    int T;
    char* blob;
    size_t bytes;
    size_t off_h, off_qkv, off_attn, off_hm, off_xnorm[2], off_idx[4], off_miss[4], off_pred[4][2], off_stats, off_hints;
    size_t sz_h, sz_qkv, sz_attn, sz_hm, sz_xnorm, sz_idx[4], sz_pred[4], sz_stats, sz_hints;
};

static void state_layout(const afx_model* m, int T, afx_state* s) {
    using afx::align256;
    const afx_model_desc& d = m->d;
    size_t o = 0;
    auto take = [&](size_t bytes) {
        const size_t at = o;
        o += align256(bytes);
        return at;
    };
    s->sz_h = static_cast<size_t>(T) * d.hidden * 4;
    s->sz_qkv = static_cast<size_t>(T) * m->n_qkv * 4;
    s->sz_attn = static_cast<size_t>(T) * d.n_heads * d.head_dim * 2;
    s->sz_hm = static_cast<size_t>(T) * d.mlp * 2;
    s->sz_xnorm = static_cast<size_t>(T) * d.hidden * 2;
    s->off_h = take(s->sz_h);
    s->off_qkv = take(s->sz_qkv);
    s->off_attn = take(s->sz_attn);
    s->off_hm = take(s->sz_hm);
    s->off_xnorm[0] = take(s->sz_xnorm);
    s->off_xnorm[1] = take(s->sz_xnorm);
    for (int op = 0; op < 4; ++op) {
        s->sz_idx[op] = static_cast<size_t>(m->K_op[op]) * 4;
        s->sz_pred[op] = static_cast<size_t>((m->K_op[op] + 31) / 32) * 4;
        s->off_idx[op] = take(s->sz_idx[op]);
        s->off_miss[op] = take(s->sz_idx[op]);
        s->off_pred[op][0] = take(s->sz_pred[op]);
        s->off_pred[op][1] = take(s->sz_pred[op]);
    }
    s->sz_stats = static_cast<size_t>(d.n_layers) * 4 * 4 * 4;
    s->off_stats = take(s->sz_stats);
    s->sz_hints = static_cast<size_t>(d.n_layers) * 4 * AFX_MAX_T * 4;
    s->off_hints = take(s->sz_hints);
    s->bytes = o;
}

extern "C" afx_status afx_model_create(const afx_model_desc* desc, const afx_layer_desc* layers,
                                       afx_model** out) {
    using namespace afx;
    if (desc == nullptr || layers == nullptr || out == nullptr) return AFX_ERR_INVALID_ARG;
    const afx_model_desc& d = *desc;
    if (d.dtype != AFX_F16 && d.dtype != AFX_BF16) return AFX_ERR_UNSUPPORTED;
    if (d.select_mode != AFX_MODE_TOPK && d.select_mode != AFX_MODE_THRESHOLD) return AFX_ERR_UNSUPPORTED;
    if (d.head_dim != kHeadDim) return AFX_ERR_UNSUPPORTED;
    if (d.xl_mode < AFX_XL_OFF || d.xl_mode > AFX_XL_REUSE) return AFX_ERR_UNSUPPORTED;
    if (d.n_layers < 1 || d.hidden < 8 || d.mlp < 8 || d.n_heads < 1 || d.n_kv_heads < 1 || d.max_seq < 1 ||
        d.xl_depth < 0 || !(d.rms_eps >= 0.0f) || !(d.rope_theta > 0.0f))
        return AFX_ERR_INVALID_ARG;
    if (d.n_heads % d.n_kv_heads != 0 || d.n_heads / d.n_kv_heads > kAttnMaxRep) return AFX_ERR_UNSUPPORTED;
    if ((d.hidden & 7) != 0 || (d.mlp & 7) != 0) return AFX_ERR_ALIGNMENT;
    const int K_op[4] = {d.hidden, d.n_heads * d.head_dim, d.hidden, d.mlp};
    for (int l = 0; l < d.n_layers; ++l) {
        const afx_layer_desc& L = layers[l];
        // (a NULL weight pointer is allowed: the operator must then come from a host handle or 4-bit rows)
        if (L.g_attn == nullptr || L.g_mlp == nullptr || L.k_cache == nullptr || L.v_cache == nullptr)
            return AFX_ERR_INVALID_ARG;
        if (!aligned16(L.w_qkv) || !aligned16(L.w_o) || !aligned16(L.w_gu) || !aligned16(L.w_down) ||
            !aligned16(L.k_cache) || !aligned16(L.v_cache) || !aligned16(L.g_attn) || !aligned16(L.g_mlp))
            return AFX_ERR_ALIGNMENT;
        for (int op = 0; op < 4; ++op) {
            if (d.select_mode == AFX_MODE_TOPK && (L.k[op] < 0 || L.k[op] > K_op[op])) return AFX_ERR_INVALID_ARG;
            if (d.select_mode == AFX_MODE_THRESHOLD && L.tau[op] != L.tau[op]) return AFX_ERR_INVALID_ARG;
        }
    }
    afx_model* m = new (std::nothrow) afx_model();
    if (m == nullptr) return AFX_ERR_CAPACITY;
    m->d = d;
    m->layers.assign(layers, layers + d.n_layers);
    m->n_qkv = (d.n_heads + 2 * d.n_kv_heads) * d.head_dim;
    for (int op = 0; op < 4; ++op) m->K_op[op] = K_op[op];
    // rotary table in fp64 on the host, stored as fp32
    const int half = kHeadDim / 2;
    std::vector<float> tab(static_cast<size_t>(2) * d.max_seq * half);
    for (int p = 0; p < d.max_seq; ++p)
        for (int i = 0; i < half; ++i) {
            const double ang = static_cast<double>(p) * pow(static_cast<double>(d.rope_theta), -2.0 * i / kHeadDim);
            tab[static_cast<size_t>(p) * half + i] = static_cast<float>(cos(ang));
            tab[static_cast<size_t>(d.max_seq + p) * half + i] = static_cast<float>(sin(ang));
        }
    if (cudaMalloc(&m->rope, tab.size() * sizeof(float)) != cudaSuccess ||
        cudaMemcpy(m->rope, tab.data(), tab.size() * sizeof(float), cudaMemcpyHostToDevice) != cudaSuccess) {
        cudaGetLastError();
        if (m->rope != nullptr) cudaFree(m->rope);
        delete m;
        return AFX_ERR_CUDA;
    }
    *out = m;
    return AFX_OK;
}

extern "C" afx_status afx_model_destroy(afx_model* model) {
    if (model == nullptr) return AFX_ERR_INVALID_ARG;
    if (model->rope != nullptr) cudaFree(model->rope);
    delete model;
    return AFX_OK;
}

extern "C" size_t afx_state_bytes(const afx_model* model, int T) {
    if (model == nullptr || T < 1 || T > AFX_MAX_T) return 0;
    afx_state s;
    state_layout(model, T, &s);
    return s.bytes;
}

extern "C" afx_status afx_state_create(const afx_model* model, int T, void* blob, size_t bytes, void* stream,
                                       afx_state** out) {
    if (model == nullptr || blob == nullptr || out == nullptr || T < 1 || T > AFX_MAX_T) return AFX_ERR_INVALID_ARG;
    if ((reinterpret_cast<uintptr_t>(blob) & 255u) != 0) return AFX_ERR_ALIGNMENT;
    afx_state* s = new (std::nothrow) afx_state();
    if (s == nullptr) return AFX_ERR_CAPACITY;
    state_layout(model, T, s);
    if (bytes < s->bytes) {
        delete s;
        return AFX_ERR_CAPACITY;
    }
    // the widest input stage must fit one block's shared memory
    const size_t dyn_max = afx::fused_dyn_smem(
        afx::IN_NORM, model->d.hidden, T,
        T > 4 ? sizeof(afx::MtSmem<afx::FusedMtCap<8>::value, afx::kFusedMtStagesSmall, afx::kFusedMtRows>)
              : (T > 1 ? sizeof(afx::MtSmem<afx::FusedMtCap<4>::value, afx::kFusedMtStagesSmall, afx::kFusedMtRows>) : 0));
    if (dyn_max > afx::kMaxDynSmem || model->d.mlp > afx::kSelectFastMaxK ||
        model->d.n_heads * model->d.head_dim > afx::kSelectFastMaxK) {
        delete s;
        return AFX_ERR_UNSUPPORTED;
    }
    s->model = model;
    s->T = T;
    s->blob = static_cast<char*>(blob);
    if (cudaMemsetAsync(blob, 0, s->bytes, static_cast<cudaStream_t>(stream)) != cudaSuccess) {
        cudaGetLastError();
        delete s;
        return AFX_ERR_CUDA;
    }
    *out = s;
    return AFX_OK;
}

extern "C" afx_status afx_state_destroy(afx_state* state) {
    if (state == nullptr) return AFX_ERR_INVALID_ARG;
    delete state;
    return AFX_OK;
}

extern "C" afx_status afx_state_buffer(const afx_state* s, int which, int op, void** ptr, size_t* bytes) {
    if (s == nullptr || ptr == nullptr) return AFX_ERR_INVALID_ARG;
    size_t off = 0, sz = 0;
    switch (which) {
        case AFX_BUF_H: off = s->off_h; sz = s->sz_h; break;
        case AFX_BUF_QKV: off = s->off_qkv; sz = s->sz_qkv; break;
        case AFX_BUF_ATTN: off = s->off_attn; sz = s->sz_attn; break;
        case AFX_BUF_HM: off = s->off_hm; sz = s->sz_hm; break;
        case AFX_BUF_XNORM:
            if (op != AFX_OP_QKV && op != AFX_OP_GU) return AFX_ERR_INVALID_ARG;
            off = s->off_xnorm[op == AFX_OP_QKV ? 0 : 1]; sz = s->sz_xnorm; break;
        case AFX_BUF_IDX:
            if (op < 0 || op > 3) return AFX_ERR_INVALID_ARG;
            off = s->off_idx[op]; sz = s->sz_idx[op]; break;
        case AFX_BUF_MISS:
            if (op < 0 || op > 3) return AFX_ERR_INVALID_ARG;
            off = s->off_miss[op]; sz = s->sz_idx[op]; break;
        case AFX_BUF_STATS: off = s->off_stats; sz = s->sz_stats; break;
        case AFX_BUF_HINTS: off = s->off_hints; sz = s->sz_hints; break;
        default: return AFX_ERR_INVALID_ARG;
    }
    *ptr = s->blob + off;
    if (bytes != nullptr) *bytes = sz;
    return AFX_OK;
}

namespace afx {

// Fills the selection part of a fused-op launch for operator input `op` of `layer`.
static void plan_selection(const afx_model* m, const afx_state* s, int layer, int op, bool cross_layer,
                           FusedArgs* a) {
    const afx_model_desc& d = m->d;
    const afx_layer_desc& L = m->layers[layer];
    int32_t* stats = reinterpret_cast<int32_t*>(s->blob + s->off_stats);
    int32_t* my_stats = stats + (static_cast<size_t>(layer) * 4 + op) * 4;
    a->mode = d.select_mode;
    a->k = L.k[op];
    a->tau = L.tau[op];
    a->idx_in = nullptr;
    a->count_in = nullptr;
    a->idx_out = reinterpret_cast<int32_t*>(s->blob + s->off_idx[op]);
    a->count_out = my_stats + 0;
    a->bitmap_out = nullptr;
    a->bitmap_pred = nullptr;
    a->miss_out = nullptr;
    a->miss_count = nullptr;
    a->hit_count = nullptr;
    a->kth_slot = my_stats + 3;
    a->kth_multi = reinterpret_cast<int32_t*>(s->blob + s->off_hints) + (static_cast<size_t>(layer) * 4 + op) * AFX_MAX_T;
    const int depth = d.xl_depth;
    if (!cross_layer || depth <= 0 || d.xl_mode == AFX_XL_OFF) return;
    const bool predictor = (layer % depth) == 0;
    const bool predicted = layer > 0;
    const int p = predicted ? depth * ((layer - 1) / depth) : 0;  // the layer whose set predicts this one
    if (predicted && !predictor && d.xl_mode == AFX_XL_REUSE) {
        a->idx_in = a->idx_out;  // the predictor's list, still in place
        a->count_in = stats + (static_cast<size_t>(p) * 4 + op) * 4;
        a->idx_out = nullptr;
        return;
    }
    if (predicted) {
        a->bitmap_pred = reinterpret_cast<const uint32_t*>(s->blob + s->off_pred[op][(p / depth) & 1]);
        a->miss_out = reinterpret_cast<int32_t*>(s->blob + s->off_miss[op]);
        a->hit_count = my_stats + 1;
        a->miss_count = my_stats + 2;
    }
    if (predictor) a->bitmap_out = reinterpret_cast<uint32_t*>(s->blob + s->off_pred[op][(layer / depth) & 1]);
}

static afx_status check_step(const afx_model* m, int layer, const afx_state* s) {
    if (m == nullptr || s == nullptr) return AFX_ERR_INVALID_ARG;
    if (s->model != m) return AFX_ERR_INVALID_ARG;
    if (layer < 0 || layer >= m->d.n_layers) return AFX_ERR_INVALID_ARG;
    return AFX_OK;
}

}  // namespace afx

namespace afx {

// One of the five kernels of a layer step (which = AFX_STEP_*), on validated arguments.
static afx_status launch_layer_kernel(afx_model* m, int layer, afx_state* s, int pos, int which, cudaStream_t st) {
    const afx_model_desc& d = m->d;
    const afx_layer_desc& L = m->layers[layer];
    float* h = reinterpret_cast<float*>(s->blob + s->off_h);
    float* qkv = reinterpret_cast<float*>(s->blob + s->off_qkv);
    uint16_t* attn = reinterpret_cast<uint16_t*>(s->blob + s->off_attn);
    uint16_t* hm = reinterpret_cast<uint16_t*>(s->blob + s->off_hm);
    const int n_attn = d.n_heads * d.head_dim;

    FusedArgs a = {};
    a.T = s->T;
    a.eps = d.rms_eps;
    switch (which) {
        case AFX_STEP_QKV:  // q | k | v
            if (L.w_qkv == nullptr) return AFX_ERR_INVALID_ARG;
            a.Wt = static_cast<const uint16_t*>(L.w_qkv);
            a.ldw = m->n_qkv;
            a.K = d.hidden;
            a.N = m->n_qkv;
            a.h = h;
            a.gain = L.g_attn;
            a.xnorm_out = reinterpret_cast<uint16_t*>(s->blob + s->off_xnorm[0]);
            a.ep = {qkv, nullptr, m->n_qkv};
            plan_selection(m, s, layer, AFX_OP_QKV, true, &a);
            return launch_fused<IN_NORM, EP_STORE>(d.dtype, a, st);
        case AFX_STEP_ATTN: {  // rotary, cache append, dense attention
            AttnArgs at = {};
            at.qkv = qkv;
            at.n_qkv = m->n_qkv;
            at.q_heads = d.n_heads;
            at.kv_heads = d.n_kv_heads;
            at.T = s->T;
            at.k_cache = static_cast<uint16_t*>(L.k_cache);
            at.v_cache = static_cast<uint16_t*>(L.v_cache);
            at.max_seq = d.max_seq;
            at.pos = pos;
            at.rope_cos = m->rope;
            at.rope_sin = m->rope + static_cast<size_t>(d.max_seq) * (kHeadDim / 2);
            at.out = attn;
            return launch_attention(d.dtype, at, st);
        }
        case AFX_STEP_O:
            if (L.w_o == nullptr) return AFX_ERR_INVALID_ARG;
            a.Wt = static_cast<const uint16_t*>(L.w_o);
            a.ldw = d.hidden;
            a.K = n_attn;
            a.N = d.hidden;
            a.x = attn;
            a.ep = {h, nullptr, d.hidden};
            plan_selection(m, s, layer, AFX_OP_O, true, &a);
            return launch_fused<IN_X, EP_ACCUM>(d.dtype, a, st);
        case AFX_STEP_GU:  // gate | up, silu(gate) * up
            if (L.w_gu == nullptr) return AFX_ERR_INVALID_ARG;
            a.Wt = static_cast<const uint16_t*>(L.w_gu);
            a.ldw = 2 * static_cast<int64_t>(d.mlp);
            a.K = d.hidden;
            a.N = 2 * d.mlp;
            a.h = h;
            a.gain = L.g_mlp;
            a.xnorm_out = reinterpret_cast<uint16_t*>(s->blob + s->off_xnorm[1]);
            a.ep = {nullptr, hm, 2 * d.mlp};
            plan_selection(m, s, layer, AFX_OP_GU, true, &a);
            return launch_fused<IN_NORM, EP_SILU>(d.dtype, a, st);
        case AFX_STEP_DOWN:
            if (L.w_down == nullptr) return AFX_ERR_INVALID_ARG;
            a.Wt = static_cast<const uint16_t*>(L.w_down);
            a.ldw = d.hidden;
            a.K = d.mlp;
            a.N = d.hidden;
            a.x = hm;
            a.ep = {h, nullptr, d.hidden};
            plan_selection(m, s, layer, AFX_OP_DOWN, true, &a);
            return launch_fused<IN_X, EP_ACCUM>(d.dtype, a, st);
        default: return AFX_ERR_INVALID_ARG;
    }
}

}  // namespace afx

extern "C" afx_status afx_layer_step(afx_model* m, int layer, afx_state* s, int pos, void* stream) {
    using namespace afx;
    afx_status rc = check_step(m, layer, s);
    if (rc != AFX_OK) return rc;
    if (pos < 0 || pos >= m->d.max_seq) return AFX_ERR_INVALID_ARG;
    for (int which = AFX_STEP_QKV; which <= AFX_STEP_DOWN; ++which)
        if ((rc = launch_layer_kernel(m, layer, s, pos, which, static_cast<cudaStream_t>(stream))) != AFX_OK) return rc;
    return AFX_OK;
}

extern "C" afx_status afx_layer_kernel(afx_model* m, int layer, afx_state* s, int pos, int which, void* stream) {
    using namespace afx;
    afx_status rc = check_step(m, layer, s);
    if (rc != AFX_OK) return rc;
    if (pos < 0 || pos >= m->d.max_seq || which < AFX_STEP_QKV || which > AFX_STEP_DOWN) return AFX_ERR_INVALID_ARG;
    return launch_layer_kernel(m, layer, s, pos, which, static_cast<cudaStream_t>(stream));
}

namespace afx {

// Input stage + selection of one operator WITHOUT its GEMV: one block that writes what a fused
// launch's side-output block writes (normed input, active list, count, cross-layer bookkeeping).
template <int IN>
static afx_status launch_select_only(int dtype, const FusedArgs& a, cudaStream_t st) {
    FusedArgs b = a;
    b.side_cluster = 1;
    b.N = 8;  // no column tile is streamed: the grid holds the side-output cluster only
    const size_t dyn = fused_dyn_smem(IN, a.K, a.T);
    auto go = [&](auto kern) { return launch_clustered(kern, 1, 1, dyn, b, st); };
    if (dtype == AFX_F16) {
        if (a.T <= 1) return go(fused_op_kernel<AFX_F16, 1, 64, IN, EP_STORE>);
        if (a.T <= 4) return go(fused_op_kernel<AFX_F16, 4, 64, IN, EP_STORE>);
        return go(fused_op_kernel<AFX_F16, 8, 64, IN, EP_STORE>);
    }
    if (a.T <= 1) return go(fused_op_kernel<AFX_BF16, 1, 64, IN, EP_STORE>);
    if (a.T <= 4) return go(fused_op_kernel<AFX_BF16, 4, 64, IN, EP_STORE>);
    return go(fused_op_kernel<AFX_BF16, 8, 64, IN, EP_STORE>);
}

}  // namespace afx

extern "C" afx_status afx_layer_step_hosted(afx_model* m, int layer, afx_state* s, int pos, const afx_hosted_ops* ops,
                                            int32_t* dev_status, void* stream) {
    using namespace afx;
    afx_status rc = check_step(m, layer, s);
    if (rc != AFX_OK) return rc;
    if (ops == nullptr || pos < 0 || pos >= m->d.max_seq) return AFX_ERR_INVALID_ARG;
    if (m->d.xl_mode == AFX_XL_REUSE) return AFX_ERR_UNSUPPORTED;  // a hosted operator always selects for itself
    const afx_model_desc& d = m->d;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    const int N_op[4] = {m->n_qkv, d.hidden, 2 * d.mlp, d.hidden};
    for (int op = 0; op < 4; ++op) {
        const bool hosted = ops->cache[op] != nullptr || ops->swap[op] != nullptr;
        if (ops->cache[op] != nullptr && ops->swap[op] != nullptr) return AFX_ERR_INVALID_ARG;
        if (hosted && (ops->slot[op] == nullptr || (reinterpret_cast<uintptr_t>(ops->slot[op]) & 3u) != 0))
            return ops->slot[op] == nullptr ? AFX_ERR_INVALID_ARG : AFX_ERR_ALIGNMENT;
        if (hosted) {
            const HostedRows r = ops->cache[op] != nullptr ? cache_rows(ops->cache[op]) : swap_rows(ops->swap[op]);
            if (r.K != m->K_op[op] || r.N != N_op[op]) return AFX_ERR_INVALID_ARG;
        }
    }
    float* h = reinterpret_cast<float*>(s->blob + s->off_h);
    float* qkv = reinterpret_cast<float*>(s->blob + s->off_qkv);
    uint16_t* attn = reinterpret_cast<uint16_t*>(s->blob + s->off_attn);
    uint16_t* hm = reinterpret_cast<uint16_t*>(s->blob + s->off_hm);
    int32_t* stats = reinterpret_cast<int32_t*>(s->blob + s->off_stats);
    const afx_layer_desc& L = m->layers[layer];
    const int which_of[4] = {AFX_STEP_QKV, AFX_STEP_O, AFX_STEP_GU, AFX_STEP_DOWN};
    for (int op = 0; op < 4; ++op) {
        if (op == AFX_OP_O && (rc = launch_layer_kernel(m, layer, s, pos, AFX_STEP_ATTN, st)) != AFX_OK) return rc;
        if (ops->cache[op] == nullptr && ops->swap[op] == nullptr) {  // resident weights: the fused kernel
            if ((rc = launch_layer_kernel(m, layer, s, pos, which_of[op], st)) != AFX_OK) return rc;
            continue;
        }
        // 1. input stage + selection
        FusedArgs a = {};
        a.T = s->T;
        a.eps = d.rms_eps;
        a.K = m->K_op[op];
        a.ldw = N_op[op];
        const uint16_t* x16 = nullptr;  // the operator's 16-bit input
        const bool norm = op == AFX_OP_QKV || op == AFX_OP_GU;
        if (norm) {
            a.h = h;
            a.gain = op == AFX_OP_QKV ? L.g_attn : L.g_mlp;
            a.xnorm_out = reinterpret_cast<uint16_t*>(s->blob + s->off_xnorm[op == AFX_OP_QKV ? 0 : 1]);
            x16 = a.xnorm_out;
        } else {
            a.x = op == AFX_OP_O ? attn : hm;
            x16 = a.x;
        }
        plan_selection(m, s, layer, op, true, &a);
        rc = norm ? launch_select_only<IN_NORM>(d.dtype, a, st) : launch_select_only<IN_X>(d.dtype, a, st);
        if (rc != AFX_OK) return rc;
        const int32_t* idx = a.idx_out;
        const int32_t* count = stats + (static_cast<size_t>(layer) * 4 + op) * 4;
        // 2. where the active columns are (fetching what is missing)
        GemvListArgs g = {};
        if (ops->cache[op] != nullptr) {
            const HostedRows r = cache_rows(ops->cache[op]);
            g.Wt = static_cast<const uint16_t*>(r.rows);
            g.ldw = r.ldw;
            rc = afx_cache_fetch(ops->cache[op], idx, count, ops->slot[op], nullptr, dev_status, stream);
        } else {
            const void* rows = nullptr;
            g.ldw = swap_rows(ops->swap[op]).ldw;
            rc = afx_swap_acquire(ops->swap[op], layer, idx, count, ops->slot[op], nullptr, dev_status, stream, &rows);
            g.Wt = static_cast<const uint16_t*>(rows);
        }
        if (rc != AFX_OK) return rc;
        // 3. the operator on the fetched rows
        g.K = m->K_op[op];
        g.N = N_op[op];
        g.T = s->T;
        g.x = x16;
        g.idx = idx;
        g.count = count;
        g.slot = ops->slot[op];
        g.status = dev_status;
        switch (op) {
            case AFX_OP_QKV: g.ep = {qkv, nullptr, N_op[op], nullptr}; break;
            case AFX_OP_GU: g.silu = 1; g.ep = {nullptr, hm, N_op[op], nullptr}; break;
            default: g.accumulate = 1; g.ep = {h, nullptr, N_op[op], nullptr}; break;
        }
        if ((rc = launch_list_gemv(d.dtype, g, st)) != AFX_OK) return rc;
    }
    return AFX_OK;
}

extern "C" afx_status afx_layer_step_q4(afx_model* m, int layer, afx_state* s, int pos, const afx_q4_layer* q4,
                                        int32_t* dev_status, void* stream) {
    using namespace afx;
    afx_status rc = check_step(m, layer, s);
    if (rc != AFX_OK) return rc;
    if (q4 == nullptr || pos < 0 || pos >= m->d.max_seq) return AFX_ERR_INVALID_ARG;
    if (s->T != 1) return AFX_ERR_UNSUPPORTED;
    if ((reinterpret_cast<uintptr_t>(dev_status) & 3u) != 0) return AFX_ERR_ALIGNMENT;
    (void)dev_status;  // every list this path multiplies by comes from its own selection: nothing to report
    const afx_model_desc& d = m->d;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    const int N_op[4] = {m->n_qkv, d.hidden, 2 * d.mlp, d.hidden};
    for (int op = 0; op < 4; ++op) {
        if (q4->wq[op] == nullptr) continue;
        if ((N_op[op] & 31) != 0) return AFX_ERR_UNSUPPORTED;
        if (!aligned16(q4->wq[op]) || (q4->ldq_bytes[op] & 15) != 0) return AFX_ERR_ALIGNMENT;
        if (q4->ldq_bytes[op] < static_cast<int64_t>(afx_q4_row_bytes(N_op[op]))) return AFX_ERR_INVALID_ARG;
    }
    float* h = reinterpret_cast<float*>(s->blob + s->off_h);
    float* qkv = reinterpret_cast<float*>(s->blob + s->off_qkv);
    uint16_t* attn = reinterpret_cast<uint16_t*>(s->blob + s->off_attn);
    uint16_t* hm = reinterpret_cast<uint16_t*>(s->blob + s->off_hm);
    const afx_layer_desc& L = m->layers[layer];
    const int which_of[4] = {AFX_STEP_QKV, AFX_STEP_O, AFX_STEP_GU, AFX_STEP_DOWN};
    for (int op = 0; op < 4; ++op) {
        if (op == AFX_OP_O && (rc = launch_layer_kernel(m, layer, s, pos, AFX_STEP_ATTN, st)) != AFX_OK) return rc;
        if (q4->wq[op] == nullptr) {  // 16-bit weights: the fused kernel
            if ((rc = launch_layer_kernel(m, layer, s, pos, which_of[op], st)) != AFX_OK) return rc;
            continue;
        }
        // input stage + selection + the operator on the 4-bit rows of the active channels, one kernel
        FusedArgs a = {};
        a.T = 1;
        a.eps = d.rms_eps;
        a.Wt = static_cast<const uint16_t*>(q4->wq[op]);
        a.ldw = q4->ldq_bytes[op] >> 1;
        a.K = m->K_op[op];
        a.N = N_op[op];
        plan_selection(m, s, layer, op, true, &a);
        switch (op) {
            case AFX_OP_QKV:
                a.h = h;
                a.gain = L.g_attn;
                a.xnorm_out = reinterpret_cast<uint16_t*>(s->blob + s->off_xnorm[0]);
                a.ep = {qkv, nullptr, N_op[op]};
                rc = launch_fused_q4<IN_NORM, EP_STORE>(d.dtype, a, st);
                break;
            case AFX_OP_GU:
                a.h = h;
                a.gain = L.g_mlp;
                a.xnorm_out = reinterpret_cast<uint16_t*>(s->blob + s->off_xnorm[1]);
                a.ep = {nullptr, hm, N_op[op]};
                rc = launch_fused_q4<IN_NORM, EP_SILU>(d.dtype, a, st);
                break;
            default:
                a.x = op == AFX_OP_O ? attn : hm;
                a.ep = {h, nullptr, N_op[op]};
                rc = launch_fused_q4<IN_X, EP_ACCUM>(d.dtype, a, st);
                break;
        }
        if (rc != AFX_OK) return rc;
    }
    return AFX_OK;
}

extern "C" afx_status afx_mlp_block(afx_model* m, int layer, afx_state* s, const void* x, float* y,
                                    void* stream) {
    using namespace afx;
    afx_status rc = check_step(m, layer, s);
    if (rc != AFX_OK) return rc;
    if (x == nullptr || y == nullptr) return AFX_ERR_INVALID_ARG;
    if ((reinterpret_cast<uintptr_t>(x) & 1u) != 0 || !aligned16(y)) return AFX_ERR_ALIGNMENT;
    const afx_model_desc& d = m->d;
    const afx_layer_desc& L = m->layers[layer];
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    uint16_t* hm = reinterpret_cast<uint16_t*>(s->blob + s->off_hm);
    if (L.w_gu == nullptr || L.w_down == nullptr) return AFX_ERR_INVALID_ARG;
    FusedArgs a = {};
    a.T = s->T;
    a.eps = d.rms_eps;
    a.Wt = static_cast<const uint16_t*>(L.w_gu);
    a.ldw = 2 * static_cast<int64_t>(d.mlp);
    a.K = d.hidden;
    a.N = 2 * d.mlp;
    a.x = static_cast<const uint16_t*>(x);
    a.ep = {nullptr, hm, 2 * d.mlp};
    plan_selection(m, s, layer, AFX_OP_GU, false, &a);
    if ((rc = launch_fused<IN_X, EP_SILU>(d.dtype, a, st)) != AFX_OK) return rc;
    a.Wt = static_cast<const uint16_t*>(L.w_down);
    a.ldw = d.hidden;
    a.K = d.mlp;
    a.N = d.hidden;
    a.x = hm;
    a.ep = {y, nullptr, d.hidden};
    plan_selection(m, s, layer, AFX_OP_DOWN, false, &a);
    return launch_fused<IN_X, EP_STORE>(d.dtype, a, st);
}

extern "C" afx_status afx_select_gemv(const void* Wt, int dtype, int K, int N, int64_t ldw, const void* x, int T,
                                      int mode, int k, float tau, float* y, int accumulate, int32_t* idx_out,
                                      int32_t* count_out, int32_t* kth_hint, void* stream) {
    using namespace afx;
    if (Wt == nullptr || x == nullptr || y == nullptr) return AFX_ERR_INVALID_ARG;
    if (K <= 0 || N <= 0 || T < 1 || T > AFX_MAX_T || ldw < N) return AFX_ERR_INVALID_ARG;
    if (K > kSelectFastMaxK) return AFX_ERR_CAPACITY;
    if (dtype != AFX_F16 && dtype != AFX_BF16) return AFX_ERR_UNSUPPORTED;
    if (mode != AFX_MODE_TOPK && mode != AFX_MODE_THRESHOLD) return AFX_ERR_UNSUPPORTED;
    if (mode == AFX_MODE_TOPK && (k < 0 || k > K)) return AFX_ERR_INVALID_ARG;
    if (mode == AFX_MODE_THRESHOLD && tau != tau) return AFX_ERR_INVALID_ARG;
    if ((N & 7) != 0 || (ldw & 7) != 0 || !aligned16(Wt) || !aligned16(y) ||
        (reinterpret_cast<uintptr_t>(x) & 1u) != 0 || (reinterpret_cast<uintptr_t>(idx_out) & 3u) != 0 ||
        (reinterpret_cast<uintptr_t>(count_out) & 3u) != 0 || (reinterpret_cast<uintptr_t>(kth_hint) & 3u) != 0)
        return AFX_ERR_ALIGNMENT;
    if ((N + 63) / 64 > 65535) return AFX_ERR_CAPACITY;
    FusedArgs a = {};
    a.Wt = static_cast<const uint16_t*>(Wt);
    a.ldw = ldw;
    a.K = K;
    a.N = N;
    a.T = T;
    a.x = static_cast<const uint16_t*>(x);
    a.mode = mode;
    a.k = k;
    a.tau = tau;
    a.ep = {y, nullptr, N};
    a.idx_out = idx_out;
    a.count_out = count_out;
    a.kth_slot = kth_hint;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    return accumulate ? launch_fused<IN_X, EP_ACCUM>(dtype, a, st) : launch_fused<IN_X, EP_STORE>(dtype, a, st);
}

// ---------------------------------------------------------------------------------------------
// afx_moe_block: dense router + the chosen experts' sparse MLP blocks (Mixtral-shaped layers).
// ---------------------------------------------------------------------------------------------

namespace afx {

constexpr int kMoeMaxExperts = 16;
constexpr int kMoeMaxTop = 4;
constexpr int kMoeThreads = 1024;

struct MoeWork {  // layout of the caller's workspace
    float logits[kMoeMaxExperts];
    int32_t sel[kMoeMaxTop];
    float weight[kMoeMaxTop];
};

// logits = W_r x over all channels (fp32, fixed order: a thread's channels ascending, lanes by
// shuffle, warps in warp order), the `top` largest (ties to the lower expert id), softmax over
// the chosen logits.  One block.
template <int DT>
__global__ void __launch_bounds__(kMoeThreads, 1)
moe_router_kernel(const uint16_t* __restrict__ x, const uint16_t* __restrict__ Wr, int64_t ldr, int K, int E, int top,
                  MoeWork* __restrict__ w) {
    __shared__ float part[kMoeThreads / 32][kMoeMaxExperts];
    float acc[kMoeMaxExperts];
#pragma unroll
    for (int e = 0; e < kMoeMaxExperts; ++e) acc[e] = 0.0f;
    for (int j = threadIdx.x; j < K; j += kMoeThreads) {
        const float xv = bits_to_float<DT>(x[j]);
        const uint16_t* row = Wr + static_cast<int64_t>(j) * ldr;
#pragma unroll
        for (int e = 0; e < kMoeMaxExperts; ++e)
            if (e < E) acc[e] = fmaf(xv, bits_to_float<DT>(row[e]), acc[e]);
    }
#pragma unroll
    for (int e = 0; e < kMoeMaxExperts; ++e) {
        const float v = warp_sum(acc[e]);
        if (lane_id() == 0) part[warp_id()][e] = v;
    }
    __syncthreads();
    if (threadIdx.x == 0) {
        float lg[kMoeMaxExperts];
        for (int e = 0; e < E; ++e) {
            float s = 0.0f;
            for (int g = 0; g < kMoeThreads / 32; ++g) s += part[g][e];
            lg[e] = s;
            w->logits[e] = s;
        }
        uint32_t taken = 0;
        float chosen[kMoeMaxTop];
        for (int r = 0; r < top; ++r) {
            int best = -1;
            for (int e = 0; e < E; ++e)
                if (!((taken >> e) & 1u) && (best < 0 || lg[e] > lg[best])) best = e;  // strict >: the lower id wins a tie
            taken |= 1u << best;
            w->sel[r] = best;
            chosen[r] = lg[best];
        }
        float z = 0.0f, p[kMoeMaxTop];
        for (int r = 0; r < top; ++r) {
            p[r] = expf(chosen[r] - chosen[0]);
            z += p[r];
        }
        for (int r = 0; r < top; ++r) w->weight[r] = p[r] / z;
    }
}

// y[i] (+)= sum over the chosen experts r, in order, of their weighted down projections part[r][i].
__global__ void __launch_bounds__(256) moe_combine_kernel(const float* __restrict__ part, int64_t stride, int top, int n,
                                                          int accumulate, float* __restrict__ y) {
    const int i = blockIdx.x * blockDim.x + threadIdx.x;
    if (i >= n) return;
    float s = accumulate ? y[i] : 0.0f;
    for (int r = 0; r < top; ++r) s += part[r * stride + i];
    y[i] = s;
}

static size_t moe_hm_stride(const afx_moe_desc& d) { return align256(static_cast<size_t>(d.mlp) * 2); }      // bytes
static size_t moe_part_stride(const afx_moe_desc& d) { return align256(static_cast<size_t>(d.hidden) * 4); }  // bytes

}  // namespace afx

extern "C" size_t afx_moe_workspace_bytes(const afx_moe_desc* d) {
    if (d == nullptr || d->mlp < 8 || d->top < 1 || d->top > afx::kMoeMaxTop) return 0;
    if (d->hidden < 8) return 0;
    return afx::align256(sizeof(afx::MoeWork)) + static_cast<size_t>(d->top) * (afx::moe_hm_stride(*d) + afx::moe_part_stride(*d));
}

extern "C" afx_status afx_moe_block(const afx_moe_desc* desc, const void* x, float* y, int accumulate, void* workspace,
                                    size_t workspace_bytes, void* stream) {
    using namespace afx;
    if (desc == nullptr || x == nullptr || y == nullptr || workspace == nullptr) return AFX_ERR_INVALID_ARG;
    const afx_moe_desc& d = *desc;
    if (d.w_router == nullptr || d.w_gu_table == nullptr || d.w_down_table == nullptr) return AFX_ERR_INVALID_ARG;
    if (d.hidden < 8 || d.mlp < 8 || d.n_experts < 1 || d.top < 1 || d.top > d.n_experts || d.ld_router < d.n_experts)
        return AFX_ERR_INVALID_ARG;
    if (d.n_experts > kMoeMaxExperts || d.top > kMoeMaxTop || d.hidden > kSelectFastMaxK || d.mlp > kSelectFastMaxK)
        return AFX_ERR_CAPACITY;
    if (d.dtype != AFX_F16 && d.dtype != AFX_BF16) return AFX_ERR_UNSUPPORTED;
    if (d.select_mode != AFX_MODE_TOPK && d.select_mode != AFX_MODE_THRESHOLD) return AFX_ERR_UNSUPPORTED;
    if (d.select_mode == AFX_MODE_TOPK && (d.k_gu < 0 || d.k_gu > d.hidden || d.k_down < 0 || d.k_down > d.mlp))
        return AFX_ERR_INVALID_ARG;
    if (d.select_mode == AFX_MODE_THRESHOLD && (d.tau_gu != d.tau_gu || d.tau_down != d.tau_down)) return AFX_ERR_INVALID_ARG;
    if ((d.hidden & 7) != 0 || (d.mlp & 7) != 0 || !aligned16(y) || (reinterpret_cast<uintptr_t>(x) & 1u) != 0 ||
        (reinterpret_cast<uintptr_t>(d.w_router) & 1u) != 0 || (reinterpret_cast<uintptr_t>(d.w_gu_table) & 7u) != 0 ||
        (reinterpret_cast<uintptr_t>(d.w_down_table) & 7u) != 0 || (reinterpret_cast<uintptr_t>(workspace) & 255u) != 0)
        return AFX_ERR_ALIGNMENT;
    if (workspace_bytes < afx_moe_workspace_bytes(desc)) return AFX_ERR_CAPACITY;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    MoeWork* w = static_cast<MoeWork*>(workspace);
    char* hm_base = static_cast<char*>(workspace) + align256(sizeof(MoeWork));
    const uint16_t* xb = static_cast<const uint16_t*>(x);
    const uint16_t* wr = static_cast<const uint16_t*>(d.w_router);
    if (d.dtype == AFX_F16)
        moe_router_kernel<AFX_F16><<<1, kMoeThreads, 0, st>>>(xb, wr, d.ld_router, d.hidden, d.n_experts, d.top, w);
    else
        moe_router_kernel<AFX_BF16><<<1, kMoeThreads, 0, st>>>(xb, wr, d.ld_router, d.hidden, d.n_experts, d.top, w);
    if (cudaGetLastError() != cudaSuccess) return AFX_ERR_CUDA;
    // the chosen experts' gate | up operators in one grid (the same input, one silu(gate) * up vector each)
    float* part = reinterpret_cast<float*>(hm_base + static_cast<size_t>(d.top) * moe_hm_stride(d));
    afx_status rc;
    FusedArgs a = {};
    a.T = 1;
    a.mode = d.select_mode;
    a.wt_sel = &w->sel[0];
    a.groups = d.top;
    a.wt_table = reinterpret_cast<const uint16_t* const*>(d.w_gu_table);
    a.ldw = 2 * static_cast<int64_t>(d.mlp);
    a.K = d.hidden;
    a.N = 2 * d.mlp;
    a.x = xb;
    a.x_stride = 0;
    a.k = d.k_gu;
    a.tau = d.tau_gu;
    a.ep = {nullptr, reinterpret_cast<uint16_t*>(hm_base), 2 * d.mlp, nullptr};
    a.out_stride = static_cast<int64_t>(moe_hm_stride(d) / 2);
    if ((rc = launch_fused_family<IN_X, EP_SILU>(d.dtype, a, st)) != AFX_OK) return rc;
    // their down projections in one grid, each on the active channels of its own input and
    // weighted by its routing weight, into one partial output per expert
    a.wt_table = reinterpret_cast<const uint16_t* const*>(d.w_down_table);
    a.ldw = d.hidden;
    a.K = d.mlp;
    a.N = d.hidden;
    a.x = reinterpret_cast<const uint16_t*>(hm_base);
    a.x_stride = static_cast<int64_t>(moe_hm_stride(d) / 2);
    a.k = d.k_down;
    a.tau = d.tau_down;
    a.ep = {part, nullptr, d.hidden, &w->weight[0]};
    a.out_stride = static_cast<int64_t>(moe_part_stride(d) / 4);
    if ((rc = launch_fused_family<IN_X, EP_STORE>(d.dtype, a, st)) != AFX_OK) return rc;
    // the experts' contributions meet in the order of the router's choice
    moe_combine_kernel<<<(d.hidden + 255) / 256, 256, 0, st>>>(part, a.out_stride, d.top, d.hidden, accumulate ? 1 : 0, y);
    if (cudaGetLastError() != cudaSuccess) return AFX_ERR_CUDA;
    return AFX_OK;
}

// ---------------------------------------------------------------------------------------------
// afx_mlp_block_noalloc: the MLP block for callers that cannot allocate device memory.
// ---------------------------------------------------------------------------------------------

namespace afx {

// The intermediate vector silu(gate) * up of the block, [T][mlp] 16-bit values, lives here
// instead of in a caller-allocated state blob.  Every device that loads the library holds
// these 512 KB until the process exits.  All calls share it.
constexpr int kNoAllocMaxMlp = AFX_NOALLOC_MAX_MLP;
static __device__ __align__(256) uint16_t g_noalloc_hm[AFX_MAX_T * kNoAllocMaxMlp];

// Device address of g_noalloc_hm on the current device (host code only sees a stand-in for
// the symbol; the address has to be asked for, once per device, with that device current).
// The address is cached for the life of the process: it does not survive cudaDeviceReset.
// The lookup must not run while `st` is capturing (it is not a stream operation and may
// initialise the module on the device), so a first call under capture is refused.
static afx_status noalloc_scratch(cudaStream_t st, uint16_t** out) {
    constexpr int kMaxDevices = 64;
    static std::mutex mu;
    static uint16_t* addr[kMaxDevices] = {};
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0) {
        cudaGetLastError();
        return AFX_ERR_CUDA;
    }
    if (dev >= kMaxDevices) return AFX_ERR_CAPACITY;
    std::lock_guard<std::mutex> lock(mu);
    if (addr[dev] == nullptr) {
        cudaStreamCaptureStatus cap = cudaStreamCaptureStatusNone;
        if (cudaStreamIsCapturing(st, &cap) != cudaSuccess) {
            cudaGetLastError();
            return AFX_ERR_CUDA;
        }
        if (cap != cudaStreamCaptureStatusNone) return AFX_ERR_INVALID_ARG;
        void* p = nullptr;
        if (cudaGetSymbolAddress(&p, g_noalloc_hm) != cudaSuccess || p == nullptr) {
            cudaGetLastError();
            return AFX_ERR_CUDA;
        }
        addr[dev] = static_cast<uint16_t*>(p);
    }
    *out = addr[dev];
    return AFX_OK;
}

}  // namespace afx

extern "C" afx_status afx_mlp_block_noalloc(const void* w_gu, const void* w_down, int dtype, int hidden, int mlp,
                                            const void* x, int T, int mode, int k_gu, float tau_gu, int k_down,
                                            float tau_down, float* y, void* stream) {
    using namespace afx;
    if (w_gu == nullptr || w_down == nullptr || x == nullptr || y == nullptr) return AFX_ERR_INVALID_ARG;
    if (hidden < 8 || mlp < 8 || T < 1 || T > AFX_MAX_T) return AFX_ERR_INVALID_ARG;
    if (mlp > kNoAllocMaxMlp || hidden > kSelectFastMaxK) return AFX_ERR_CAPACITY;
    if (dtype != AFX_F16 && dtype != AFX_BF16) return AFX_ERR_UNSUPPORTED;
    if (mode != AFX_MODE_TOPK && mode != AFX_MODE_THRESHOLD) return AFX_ERR_UNSUPPORTED;
    if (mode == AFX_MODE_TOPK && (k_gu < 0 || k_gu > hidden || k_down < 0 || k_down > mlp)) return AFX_ERR_INVALID_ARG;
    if (mode == AFX_MODE_THRESHOLD && (tau_gu != tau_gu || tau_down != tau_down)) return AFX_ERR_INVALID_ARG;
    if ((hidden & 7) != 0 || (mlp & 7) != 0 || !aligned16(w_gu) || !aligned16(w_down) || !aligned16(y) ||
        (reinterpret_cast<uintptr_t>(x) & 1u) != 0)
        return AFX_ERR_ALIGNMENT;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    uint16_t* hm = nullptr;
    afx_status rc = noalloc_scratch(st, &hm);
    if (rc != AFX_OK) return rc;
    // Nothing in hm has to start from zero: the first kernel writes all T * mlp values that
    // the second one reads.
    FusedArgs a = {};
    a.T = T;
    a.Wt = static_cast<const uint16_t*>(w_gu);
    a.ldw = 2 * static_cast<int64_t>(mlp);
    a.K = hidden;
    a.N = 2 * mlp;
    a.x = static_cast<const uint16_t*>(x);
    a.mode = mode;
    a.k = k_gu;
    a.tau = tau_gu;
    a.ep = {nullptr, hm, 2 * mlp};
    if ((rc = launch_fused<IN_X, EP_SILU>(dtype, a, st)) != AFX_OK) return rc;
    a.Wt = static_cast<const uint16_t*>(w_down);
    a.ldw = hidden;
    a.K = mlp;
    a.N = hidden;
    a.x = hm;
    a.k = k_down;
    a.tau = tau_down;
    a.ep = {y, nullptr, hidden};
    return launch_fused<IN_X, EP_STORE>(dtype, a, st);
}

#ifdef AFX_EXPERIMENT
// Experiment builds only (not part of the ABI): clusters of S blocks of the bf16 one-token operator (tile width pw,
// plain input of K channels, h += epilogue) that the occupancy query reports as co-resident.
extern "C" int afx_internal_max_clusters(int pw, int S, int K) {
    using namespace afx;
    const size_t dyn = fused_dyn_smem(IN_X, K, 1);
    const void* kern = pw == 256 ? reinterpret_cast<const void*>(fused_op_kernel<AFX_BF16, 1, 256, IN_X, EP_ACCUM>)
                     : pw == 128 ? reinterpret_cast<const void*>(fused_op_kernel<AFX_BF16, 1, 128, IN_X, EP_ACCUM>)
                                 : reinterpret_cast<const void*>(fused_op_kernel<AFX_BF16, 1, 64, IN_X, EP_ACCUM>);
    return max_active_clusters(kern, S, dyn);
}
#endif
