// afx_sparse_gemv: host-side shape selection and launch.
#include "afx_launch.cuh"
#include "afx_mma.cuh"

namespace afx {

template <int TMAX>
struct GemvShape {
    static constexpr int kBlocksPerSM = TMAX <= 1 ? 2 : 1;
    static constexpr int kStageCap = TMAX <= 4 ? 1024 : 512;
};

template <int DT, int TMAX, int PW>
__global__ void __launch_bounds__(kGemvThreads, GemvShape<TMAX>::kBlocksPerSM)
sparse_gemv_kernel(GemvListArgs a) {
    constexpr int CAP = GemvShape<TMAX>::kStageCap;
    __shared__ GemvSmem<TMAX, CAP> sm;
    __shared__ GemvRecv<TMAX> recv;
    gemv_list_block<DT, TMAX, PW, CAP>(a, &sm, &recv);
}

// A few tokens at once: the tensor-core kernel (afx_mma.cuh).  2048 staged entries per pass
// still leave room for two blocks per SM.
using MtListSmem = MtSmem<2048, 4>;
template <int DT>
__global__ void __launch_bounds__(kGemvThreads, 2) sparse_gemm_mt_kernel(GemvListArgs a) {
    extern __shared__ __align__(16) unsigned char mt_dyn[];
    mt_list_block<DT>(a, reinterpret_cast<MtListSmem*>(mt_dyn));
}

template <int DT>
static afx_status launch_gemm_mt(const GemvListArgs& a, cudaStream_t st) {
    const void* kern = reinterpret_cast<const void*>(sparse_gemm_mt_kernel<DT>);
    const size_t dyn = sizeof(MtListSmem);
    const int tiles = (a.N + kMtTile - 1) / kMtTile;
    if (tiles > 65535) return AFX_ERR_CAPACITY;
    // the largest cluster that keeps every tile's cluster resident at once (a margin stays free, as for the fp32 kernels)
    const int margin = (tiles + 15) / 16 < 2 ? 2 : (tiles + 15) / 16;
    int S = 1;
    for (int s = kMaxCluster; s > 1; --s)
        if (max_active_clusters(kern, s, dyn) >= tiles + margin) {
            S = s;
            break;
        }
    return launch_clustered(sparse_gemm_mt_kernel<DT>, S, tiles, dyn, a, st);
}

int sm_count() {
    static int cached[64];
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= 64) return 0;
    if (cached[dev] == 0) {
        int n = 0;
        if (cudaDeviceGetAttribute(&n, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess) return 0;
        cached[dev] = n;
    }
    return cached[dev];
}

#ifdef AFX_EXPERIMENT
int g_force_pw = 0, g_force_s = 0;  // experiment knobs, 0 = automatic
int g_cluster_margin = -1;          // experiment knob, < 0 = automatic
#endif

template <int DT, int TMAX>
static afx_status launch_gemv_t(const GemvListArgs& a, cudaStream_t st) {
    const void* kerns[3] = {reinterpret_cast<const void*>(sparse_gemv_kernel<DT, TMAX, 256>),
                            reinterpret_cast<const void*>(sparse_gemv_kernel<DT, TMAX, 128>),
                            reinterpret_cast<const void*>(sparse_gemv_kernel<DT, TMAX, 64>)};
    const GemvShapeChoice c = choose_gemv_shape(a.N, kerns, 0);
    switch (c.pw) {
        case 256: return launch_clustered(sparse_gemv_kernel<DT, TMAX, 256>, c.S, c.tiles, 0, a, st);
        case 128: return launch_clustered(sparse_gemv_kernel<DT, TMAX, 128>, c.S, c.tiles, 0, a, st);
        default: return launch_clustered(sparse_gemv_kernel<DT, TMAX, 64>, c.S, c.tiles, 0, a, st);
    }
}

template <int DT>
static afx_status launch_gemv(const GemvListArgs& a, cudaStream_t st) {
    if (a.T <= 1) return launch_gemv_t<DT, 1>(a, st);
    return launch_gemm_mt<DT>(a, st);
}

afx_status launch_list_gemv(int dtype, const GemvListArgs& a, cudaStream_t st) {
    return dtype == AFX_F16 ? launch_gemv<AFX_F16>(a, st) : launch_gemv<AFX_BF16>(a, st);
}

}  // namespace afx

#ifdef AFX_EXPERIMENT
// Experiment builds only (not part of the ABI): force tile width / cluster size / margin.
extern "C" void afx_internal_tune_gemv(int pw, int s) {
    afx::g_force_pw = pw;
    afx::g_force_s = s;
}
extern "C" void afx_internal_cluster_margin(int margin) { afx::g_cluster_margin = margin; }
#endif

extern "C" size_t afx_workspace_bytes(int K_max, int N_max, int T_max) {
    (void)K_max;
    (void)N_max;
    (void)T_max;
    return 0;  // partial sums meet in (distributed) shared memory: no entry point needs scratch
}

extern "C" afx_status afx_sparse_gemv(const void* Wt, int dtype, int K, int N, int64_t ldw,
                                      const void* x, int T, const int32_t* idx, const int32_t* count,
                                      const int32_t* slot, float* y, int accumulate, int32_t* dev_status,
                                      void* stream) {
    using namespace afx;
    if (Wt == nullptr || x == nullptr || idx == nullptr || count == nullptr || y == nullptr)
        return AFX_ERR_INVALID_ARG;
    if (K <= 0 || N <= 0 || T < 1 || T > AFX_MAX_T || ldw < N) return AFX_ERR_INVALID_ARG;
    if (dtype != AFX_F16 && dtype != AFX_BF16) return AFX_ERR_UNSUPPORTED;
    if ((N & 7) != 0 || (ldw & 7) != 0 || !aligned16(Wt) || !aligned16(y) ||
        (reinterpret_cast<uintptr_t>(x) & 1u) != 0 || (reinterpret_cast<uintptr_t>(idx) & 3u) != 0 ||
        (reinterpret_cast<uintptr_t>(count) & 3u) != 0 || (reinterpret_cast<uintptr_t>(slot) & 3u) != 0 ||
        (reinterpret_cast<uintptr_t>(dev_status) & 3u) != 0)
        return AFX_ERR_ALIGNMENT;
    if ((N + 63) / 64 > 65535) return AFX_ERR_CAPACITY;
    GemvListArgs a;
    a.Wt = static_cast<const uint16_t*>(Wt);
    a.ldw = ldw;
    a.K = K;
    a.N = N;
    a.T = T;
    a.x = static_cast<const uint16_t*>(x);
    a.idx = idx;
    a.count = count;
    a.slot = slot;
    a.accumulate = accumulate ? 1 : 0;
    a.silu = 0;
    a.ep.y = y;
    a.ep.out_bits = nullptr;
    a.ep.N = N;
    a.ep.scale = nullptr;
    a.status = dev_status;
    return launch_list_gemv(dtype, a, static_cast<cudaStream_t>(stream));
}
