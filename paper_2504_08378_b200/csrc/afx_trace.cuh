// Recording form of the stage marks, used only by timing-study builds (-DAFX_TRACE).
// AFX_TRACE_REGION(r) (thread 0, at kernel start) names the kernel kind, 0..7; AFX_MARK(i)
// then stores the SM clock of mark i (0..13) of that block into afx_trace_buf
// [region][block % 512][16]; slots 15 and 14 hold the global nanosecond timer and the SM id
// at mark 0.
#pragma once

extern __device__ long long afx_trace_buf[];

__device__ __forceinline__ int* afx_trace_region_ptr() {
    __shared__ int region;
    return &region;
}

#define AFX_TRACE_REGION(r)                                   \
    do {                                                      \
        if (threadIdx.x == 0) *afx_trace_region_ptr() = (r);  \
    } while (0)

#define AFX_MARK(i)                                                                                   \
    do {                                                                                              \
        if (threadIdx.x == 0) {                                                                       \
            const int region_ = *afx_trace_region_ptr();                                              \
            long long* slot_ = afx_trace_buf + (region_ * 512 + (blockIdx.y * gridDim.x + blockIdx.x) % 512) * 16; \
            slot_[(i)] = clock64();                                                                   \
            if ((i) == 0) {                                                                           \
                unsigned long long ns_;                                                               \
                asm volatile("mov.u64 %0, %%globaltimer;" : "=l"(ns_));                               \
                slot_[15] = static_cast<long long>(ns_);                                              \
                unsigned sm_;                                                                         \
                asm volatile("mov.u32 %0, %%smid;" : "=r"(sm_));                                      \
                slot_[14] = static_cast<long long>(sm_);                                              \
            }                                                                                         \
        }                                                                                             \
    } while (0)
