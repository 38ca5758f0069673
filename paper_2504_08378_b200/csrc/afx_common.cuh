// Shared device/host helpers of libafx (sm_100a only).
#pragma once

#include <cuda_runtime.h>
#include <cuda_fp16.h>
#include <stdint.h>

#include "afx.h"

// Stage marks for kernel timing studies: empty unless the library is built with AFX_TRACE, in
// which case afx_trace.cuh supplies the recording form.
#ifdef AFX_TRACE
#include "afx_trace.cuh"
#else
#define AFX_MARK(i) \
    do {            \
    } while (0)
#define AFX_TRACE_REGION(r) \
    do {                    \
    } while (0)
#endif

namespace afx {

constexpr int kWarp = 32;

// ---- 16-bit storage types -----------------------------------------------------------

// |x| as an integer key: for finite values the sign-cleared bit pattern orders like |x|.
__device__ __forceinline__ uint32_t mag_key(uint16_t bits) { return bits & 0x7FFFu; }

template <int DT>
__device__ __forceinline__ float bits_to_float(uint16_t bits) {
    if (DT == AFX_F16) {
        return __half2float(__ushort_as_half(bits));
    } else {
        return __uint_as_float(static_cast<uint32_t>(bits) << 16);
    }
}

// Eight packed 16-bit weights (one 128-bit load) to fp32.
template <int DT>
__device__ __forceinline__ void unpack8(const uint4& raw, float (&w)[8]) {
    const uint32_t r[4] = {raw.x, raw.y, raw.z, raw.w};
#pragma unroll
    for (int i = 0; i < 4; ++i) {
        if (DT == AFX_F16) {
            __half2 h = *reinterpret_cast<const __half2*>(&r[i]);
            float2 f = __half22float2(h);
            w[2 * i] = f.x;
            w[2 * i + 1] = f.y;
        } else {
            w[2 * i] = __uint_as_float(r[i] << 16);
            w[2 * i + 1] = __uint_as_float(r[i] & 0xFFFF0000u);
        }
    }
}

// ---- packed fp32 pairs (two-wide fused multiply-add of sm_100) ------------------------

typedef unsigned long long f32x2;  // two fp32 values in one 64-bit register pair (low, high)

__device__ __forceinline__ f32x2 pack_f32x2(float lo, float hi) {
    f32x2 r;
    asm("mov.b64 %0, {%1, %2};" : "=l"(r) : "f"(lo), "f"(hi));
    return r;
}
__device__ __forceinline__ void unpack_f32x2(f32x2 v, float& lo, float& hi) {
    asm("mov.b64 {%0, %1}, %2;" : "=f"(lo), "=f"(hi) : "l"(v));
}
// acc = a * b + acc on both halves, each exactly as a scalar fma.rn.f32.
__device__ __forceinline__ void fma_f32x2(f32x2& acc, f32x2 a, f32x2 b) {
    asm("fma.rn.f32x2 %0, %1, %2, %0;" : "+l"(acc) : "l"(a), "l"(b));
}

// Eight packed 16-bit weights (one 128-bit load) as four fp32 pairs (weights 2i, 2i+1).
template <int DT>
__device__ __forceinline__ void unpack8_pairs(const uint4& raw, f32x2 (&w)[4]) {
    const uint32_t r[4] = {raw.x, raw.y, raw.z, raw.w};
#pragma unroll
    for (int i = 0; i < 4; ++i) {
        if (DT == AFX_F16) {
            const float2 f = __half22float2(*reinterpret_cast<const __half2*>(&r[i]));
            w[i] = pack_f32x2(f.x, f.y);
        } else {
            const uint32_t lo = r[i] << 16, hi = r[i] & 0xFFFF0000u;
            asm("mov.b64 %0, {%1, %2};" : "=l"(w[i]) : "r"(lo), "r"(hi));
        }
    }
}

// Round-to-nearest-even fp32 -> 16-bit storage.
template <int DT>
__device__ __forceinline__ uint16_t float_to_bits(float v) {
    if (DT == AFX_F16) {
        return __half_as_ushort(__float2half_rn(v));
    } else {
        uint32_t u = __float_as_uint(v);
        if ((u & 0x7FFFFFFFu) > 0x7F800000u) return static_cast<uint16_t>((u >> 16) | 0x0040u);  // NaN
        u += 0x7FFFu + ((u >> 16) & 1u);
        return static_cast<uint16_t>(u >> 16);
    }
}

// ---- memory access -------------------------------------------------------------------

// 128-bit streaming read of weights: read-only path, no L1 allocation (each byte is used once).
__device__ __forceinline__ uint4 ld_stream_16B(const void* p) {
    uint4 v;
    asm volatile("ld.global.nc.L1::no_allocate.v4.u32 {%0,%1,%2,%3}, [%4];"
                 : "=r"(v.x), "=r"(v.y), "=r"(v.z), "=r"(v.w)
                 : "l"(p));
    return v;
}

// ---- warp / block primitives ---------------------------------------------------------

__host__ __device__ __forceinline__ int64_t min64(int64_t a, int64_t b) { return a < b ? a : b; }
__host__ __device__ __forceinline__ int64_t max64(int64_t a, int64_t b) { return a > b ? a : b; }

__device__ __forceinline__ int lane_id() { return threadIdx.x & 31; }
__device__ __forceinline__ int warp_id() { return threadIdx.x >> 5; }

__device__ __forceinline__ int warp_sum(int v) {
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xFFFFFFFFu, v, o);
    return v;
}

__device__ __forceinline__ float warp_sum(float v) {
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xFFFFFFFFu, v, o);
    return v;
}

// Exclusive prefix sum of one int per warp (at most 32 warps), via shared memory.
// `warp_total` is this warp's value (same in all lanes); `scratch` holds 33 ints.
// Returns this warp's exclusive prefix; scratch[32] receives the block total.
// Contains block-wide barriers: every thread of the block must call it.
__device__ __forceinline__ int block_exclusive_over_warps(int warp_total, int* scratch) {
    const int nw = (blockDim.x + 31) >> 5;
    __syncthreads();  // scratch may still be read from a previous use
    if (lane_id() == 0) scratch[warp_id()] = warp_total;
    __syncthreads();
    if (warp_id() == 0) {
        int v = lane_id() < nw ? scratch[lane_id()] : 0;
        int incl = v;
#pragma unroll
        for (int o = 1; o < 32; o <<= 1) {
            int n = __shfl_up_sync(0xFFFFFFFFu, incl, o);
            if (lane_id() >= o) incl += n;
        }
        scratch[lane_id()] = incl - v;
        if (lane_id() == 31) scratch[32] = incl;
    }
    __syncthreads();
    return scratch[warp_id()];
}

// ---- device status word ----------------------------------------------------------------

// Records the first problem a kernel met in caller-provided data (a list entry or a count out
// of range): the word keeps the first non-zero code until the caller clears it.
__device__ __forceinline__ void report_status(int32_t* status, int32_t code) {
    if (status != nullptr) atomicCAS(status, 0, code);
}

// ---- host side -----------------------------------------------------------------------

inline bool aligned16(const void* p) { return (reinterpret_cast<uintptr_t>(p) & 15u) == 0; }

inline afx_status launch_status() {
    return cudaGetLastError() == cudaSuccess ? AFX_OK : AFX_ERR_CUDA;
}

// Number of SMs of the current device (cached per device id).
int sm_count();

}  // namespace afx
