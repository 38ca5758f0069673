// afx_sparse_gemv and its workspace.
#include "afx_gemv.cuh"

namespace afx {

// Launch shapes.  512 threads per block; tokens decide the register budget and with it how
// many blocks stay resident per SM.
constexpr int kGemvWN = 1;
constexpr int kGemvWC = 16;
constexpr int kGemvThreads = 32 * kGemvWN * kGemvWC;
constexpr int kGemvUnroll = 8;
constexpr int kCountersBytes = 4096;  // room for 1024 tile counters

template <int TMAX>
struct GemvShape {
    static constexpr int kBlocksPerSM = TMAX <= 2 ? 2 : 1;
    static constexpr int kStageCap = TMAX <= 4 ? 1024 : 512;
};

template <int DT, int TMAX>
__global__ void __launch_bounds__(kGemvThreads, GemvShape<TMAX>::kBlocksPerSM)
sparse_gemv_kernel(GemvArgs a) {
    constexpr int CAP = GemvShape<TMAX>::kStageCap;
    __shared__ GemvShared<CAP> sh;
    __shared__ float s_x[TMAX * CAP];
    __shared__ __align__(16) float s_red[kGemvWC * kGemvWN * kPieceW];
    gemv_block<DT, TMAX, kGemvWN, kGemvWC, kGemvUnroll, CAP>(a, &sh, s_x, s_red);
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

static int gemv_grid(int tmax) {
    const int per_sm = tmax <= 2 ? 2 : 1;
    return sm_count() * per_sm;
}

static int tmax_for(int T) { return T <= 1 ? 1 : (T <= 2 ? 2 : (T <= 4 ? 4 : 8)); }

template <int DT>
static afx_status launch_gemv(const GemvArgs& a, cudaStream_t st) {
    const int tmax = tmax_for(a.T);
    const int grid = gemv_grid(tmax);
    if (grid <= 0) return AFX_ERR_CUDA;
    switch (tmax) {
        case 1: sparse_gemv_kernel<DT, 1><<<grid, kGemvThreads, 0, st>>>(a); break;
        case 2: sparse_gemv_kernel<DT, 2><<<grid, kGemvThreads, 0, st>>>(a); break;
        case 4: sparse_gemv_kernel<DT, 4><<<grid, kGemvThreads, 0, st>>>(a); break;
        default: sparse_gemv_kernel<DT, 8><<<grid, kGemvThreads, 0, st>>>(a); break;
    }
    return launch_status();
}

}  // namespace afx

extern "C" size_t afx_workspace_bytes(int N_max, int T_max) {
    using namespace afx;
    if (N_max <= 0 || T_max < 1 || T_max > AFX_MAX_T) return 0;
    const int sms = sm_count();
    const size_t blocks = static_cast<size_t>(sms > 0 ? sms : 256) * 2;
    const size_t tiles = static_cast<size_t>(N_max + kPieceW - 1) / kPieceW;
    if (tiles * sizeof(int) > kCountersBytes) return 0;
    return kCountersBytes + (blocks + tiles) * static_cast<size_t>(T_max) * kGemvWN * kPieceW * sizeof(float);
}

extern "C" afx_status afx_workspace_init(void* workspace, size_t bytes, void* stream) {
    if (workspace == nullptr || bytes < afx::kCountersBytes) return AFX_ERR_INVALID_ARG;
    if (cudaMemsetAsync(workspace, 0, afx::kCountersBytes, static_cast<cudaStream_t>(stream)) != cudaSuccess)
        return AFX_ERR_CUDA;
    return AFX_OK;
}

extern "C" afx_status afx_sparse_gemv(const void* Wt, int dtype, int K, int N, int64_t ldw,
                                      const void* x, int T, const int32_t* idx, const int32_t* count,
                                      const int32_t* slot, float* y, int accumulate, void* workspace,
                                      void* stream) {
    using namespace afx;
    if (Wt == nullptr || x == nullptr || idx == nullptr || count == nullptr || y == nullptr ||
        workspace == nullptr)
        return AFX_ERR_INVALID_ARG;
    if (K <= 0 || N <= 0 || T < 1 || T > AFX_MAX_T || ldw < N) return AFX_ERR_INVALID_ARG;
    if (dtype != AFX_F16 && dtype != AFX_BF16) return AFX_ERR_UNSUPPORTED;
    if ((N & 7) != 0 || (ldw & 7) != 0 || !aligned16(Wt) || !aligned16(y) ||
        (reinterpret_cast<uintptr_t>(workspace) & 255u) != 0 || (reinterpret_cast<uintptr_t>(x) & 1u) != 0)
        return AFX_ERR_ALIGNMENT;
    if (static_cast<size_t>(N + kPieceW - 1) / kPieceW * sizeof(int) > kCountersBytes) return AFX_ERR_CAPACITY;
    GemvArgs a;
    a.Wt = static_cast<const uint16_t*>(Wt);
    a.ldw = ldw;
    a.K = K;
    a.N = N;
    a.T = T;
    a.x = static_cast<const uint16_t*>(x);
    a.idx = idx;
    a.count = count;
    a.slot = slot;
    a.y = y;
    a.accumulate = accumulate ? 1 : 0;
    a.counters = static_cast<int*>(workspace);
    a.partials = reinterpret_cast<float*>(static_cast<char*>(workspace) + kCountersBytes);
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    return dtype == AFX_F16 ? launch_gemv<AFX_F16>(a, st) : launch_gemv<AFX_BF16>(a, st);
}
