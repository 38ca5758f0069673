// Arguments and launcher of the 4-bit sparse GEMV kernel (afx_q4.cu), shared with the layer
// step over 4-bit weights (afx_layer.cu).
#pragma once

#include <cuda_runtime.h>
#include <stdint.h>

#include "afx.h"

namespace afx {

enum { Q4_STORE = 0, Q4_ACCUM = 1, Q4_SILU = 2 };

struct Q4Args {
    const unsigned char* Wq;
    int64_t ldq;  // row stride in bytes (multiple of 16)
    int K, N;
    const uint16_t* x;
    const int32_t* idx;
    const int32_t* count;
    // how a finished sum leaves: Q4_STORE y[i] = sum, Q4_ACCUM y[i] += sum; Q4_SILU: every block
    // of 32 outputs is 16 "gate" outputs (the low 4 bits of its 16 bytes) and 16 "up" outputs
    // (the high 4 bits), out_bits[16 b + m] = round(silu(gate_m) * up_m) in x's 16-bit type
    int ep;
    float* y;
    uint16_t* out_bits;
    int32_t* status;
};

// x_dtype AFX_F16 / AFX_BF16; arguments already validated.
afx_status launch_q4_list(int x_dtype, const Q4Args& a, cudaStream_t st);

}  // namespace afx
