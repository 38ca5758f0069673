// Recording form of AFX_MARK, used only by timing-study builds (-DAFX_TRACE): thread 0 of
// every block stores the SM clock of mark i (0..14) into afx_trace_buf, in one of five
// regions told apart by the launch shape (256-thread blocks; 5-, 3- and other cluster widths,
// the last split by dynamic shared memory above / below 80 KB); slots 15 and 14 of a block
// hold the global nanosecond timer and the SM id at its mark 0.
#pragma once

extern __device__ long long afx_trace_buf[];
#define AFX_MARK(i)                                                                                   \
    do {                                                                                              \
        if (threadIdx.x == 0) {                                                                       \
            unsigned dyn_;                                                                            \
            asm volatile("mov.u32 %0, %%dynamic_smem_size;" : "=r"(dyn_));                            \
            const int region_ = blockDim.x == 256 ? 0 : (gridDim.x == 5 ? 1 : (gridDim.x == 3 ? 2 : (dyn_ > 80000u ? 3 : 4))); \
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
