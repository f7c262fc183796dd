// Shared device/host helpers for libdpclip (sm_100a only).
#pragma once
#include <cuda_bf16.h>
#include <cuda_runtime.h>
#include <stdint.h>

#include "dpclip.h"

namespace dpclip {

constexpr int kHeaderBytes = 256;   // status header at the start of every workspace
constexpr int kNumSMs = 148;        // B200: 2 dies x 74 SMs

__device__ __forceinline__ float to_f32(float x) { return x; }
__device__ __forceinline__ float to_f32(__nv_bfloat16 x) { return __bfloat162float(x); }

// Four consecutive elements as fp32 (pointer must be aligned to 4 elements).
__device__ __forceinline__ float4 load4(const float* p) { return *reinterpret_cast<const float4*>(p); }
__device__ __forceinline__ float4 load4(const __nv_bfloat16* p) {
    uint2 raw = *reinterpret_cast<const uint2*>(p);
    float4 v;
    v.x = __uint_as_float(raw.x << 16);
    v.y = __uint_as_float(raw.x & 0xFFFF0000u);
    v.z = __uint_as_float(raw.y << 16);
    v.w = __uint_as_float(raw.y & 0xFFFF0000u);
    return v;
}

__device__ __forceinline__ float warp_sum(float v) {
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xFFFFFFFFu, v, o);
    return v;
}

// Sum over a CTA of up to 1024 threads; result valid in thread 0.
__device__ __forceinline__ float block_sum(float v, float* smem32) {
    v = warp_sum(v);
    int lane = threadIdx.x & 31, w = threadIdx.x >> 5;
    __syncthreads();
    if (lane == 0) smem32[w] = v;
    __syncthreads();
    if (w == 0) {
        int nw = (blockDim.x + 31) >> 5;
        v = lane < nw ? smem32[lane] : 0.f;
        v = warp_sum(v);
    }
    return v;
}

// Range-checked build (-DDPCLIP_DEBUG, `python -m paper_2009_03106_b200.build --debug`): the stand-in for a
// memory checker.  DPCLIP_IN_RANGE(i, n, status) is true when 0 <= i < n; otherwise it records
// DPCLIP_ERR_RANGE in the workspace's status word and yields false, and the caller SKIPS the access -- no
// trap, the kernel runs to its end.  In the normal build it is the constant true and costs nothing.
#ifdef DPCLIP_DEBUG
__device__ __forceinline__ bool debug_range_violation(int* status) {
    if (status) atomicExch(status, (int)DPCLIP_ERR_RANGE);
    return false;
}
#define DPCLIP_IN_RANGE(i, n, status) \
    (((long long)(i) >= 0 && (long long)(i) < (long long)(n)) ? true : dpclip::debug_range_violation(status))
#else
#define DPCLIP_IN_RANGE(i, n, status) (true)
#endif

inline int ceil_div(long a, long b) { return (int)((a + b - 1) / b); }

}  // namespace dpclip
