// Element-wise parameter layers (LayerNorm gain and shift): h = gamma (.) hbar + beta.
//
// Per example the gradients are ggamma_i = sum_t zb_{i,t} (.) hbar_{i,t} and gbeta_i = sum_t zb_{i,t}
// (the sum over the positions that share the parameters is taken before the norm).  Both kernels are
// pure streaming: every element of Hbar and Zb is read once, two flops each.
//
//   elementwise_norm_kernel : CTA = (column block, example); 64 (or 32) column groups x 4 (8) row groups; the
//                             per-column sums over the example's T rows are combined in shared memory,
//                             squared and summed -> sq[i] (atomic when the width spans several CTAs).
//   elementwise_grad_kernel : CTA = (column block, row slice); every row weighted by its example's
//                             clip factor; per-column sums are added to g_scale / g_shift (zeroed by
//                             the launcher) with fire-and-forget adds.
#pragma once
#include "common.cuh"

namespace dpclip {

constexpr int EW_THREADS = 256;

// VEC consecutive elements as loaded (converted to fp32 only when used, so that a deep batch of loads
// costs few registers).
template <typename T, int VEC> struct EwRaw;
template <> struct EwRaw<float, 4> { float4 v; };
template <> struct EwRaw<float, 1> { float v; };
template <> struct EwRaw<__nv_bfloat16, 4> { uint2 v; };
template <> struct EwRaw<__nv_bfloat16, 1> { __nv_bfloat16 v; };

__device__ __forceinline__ void ew_load(const float* p, EwRaw<float, 4>& r) { r.v = *reinterpret_cast<const float4*>(p); }
__device__ __forceinline__ void ew_load(const float* p, EwRaw<float, 1>& r) { r.v = *p; }
__device__ __forceinline__ void ew_load(const __nv_bfloat16* p, EwRaw<__nv_bfloat16, 4>& r) { r.v = *reinterpret_cast<const uint2*>(p); }
__device__ __forceinline__ void ew_load(const __nv_bfloat16* p, EwRaw<__nv_bfloat16, 1>& r) { r.v = *p; }
__device__ __forceinline__ void ew_f32(const EwRaw<float, 4>& r, float (&x)[4]) { x[0] = r.v.x; x[1] = r.v.y; x[2] = r.v.z; x[3] = r.v.w; }
__device__ __forceinline__ void ew_f32(const EwRaw<float, 1>& r, float (&x)[1]) { x[0] = r.v; }
__device__ __forceinline__ void ew_f32(const EwRaw<__nv_bfloat16, 4>& r, float (&x)[4]) {
    x[0] = __uint_as_float(r.v.x << 16); x[1] = __uint_as_float(r.v.x & 0xFFFF0000u);
    x[2] = __uint_as_float(r.v.y << 16); x[3] = __uint_as_float(r.v.y & 0xFFFF0000u);
}
__device__ __forceinline__ void ew_f32(const EwRaw<__nv_bfloat16, 1>& r, float (&x)[1]) { x[0] = __bfloat162float(r.v); }

// Column sums of zb (.) hbar and of zb over rows r0 + rg, r0 + rg + RG, ... < r1 (RG row groups per CTA),
// each row weighted by its example's factor when WEIGHTED.  Batches of UNR rows: all loads first.
template <typename T, int VEC, int RG, bool WEIGHTED>
__device__ __forceinline__ void ew_accumulate(const T* __restrict__ H, long ldh, const T* __restrict__ Z, long ldz,
                                              long r0, long r1, int rows_per_example, const float* __restrict__ clip,
                                              int c0, int rg, float (&gg)[VEC], float (&gs)[VEC]) {
#pragma unroll
    for (int u = 0; u < VEC; ++u) { gg[u] = 0.f; gs[u] = 0.f; }
    constexpr int UNR = sizeof(T) == 2 ? 8 : 4;
    long r = r0 + rg;
    // example of row r and the row's position in it, advanced without divisions (and without a loop when an
    // example has at least RG rows: one predicated step)
    int e = WEIGHTED ? (int)(r / rows_per_example) : 0;
    int rem = WEIGHTED ? (int)(r - (long)e * rows_per_example) : 0;
    const bool one_step = rows_per_example >= RG;
    auto advance = [&](int by) {
        rem += by;
        if (one_step) { const bool over = rem >= rows_per_example; rem -= over ? rows_per_example : 0; e += over ? 1 : 0; }
        else while (rem >= rows_per_example) { rem -= rows_per_example; ++e; }
    };
    for (; r + (UNR - 1) * RG < r1; r += UNR * RG) {
        EwRaw<T, VEC> h[UNR], z[UNR];
        float w[UNR];
#pragma unroll
        for (int k = 0; k < UNR; ++k) {
            const long rr = r + k * RG;
            ew_load(H + (size_t)rr * ldh + c0, h[k]);
            ew_load(Z + (size_t)rr * ldz + c0, z[k]);
            w[k] = 1.f;
        }
        if (WEIGHTED) {
            // the rows of a batch are the same for the whole warp; when they lie in one example (the usual
            // case) one factor load serves the batch instead of one per row
            if (rem + (UNR - 1) * RG < rows_per_example) {
                const float w0 = __ldg(clip + e);
#pragma unroll
                for (int k = 0; k < UNR; ++k) w[k] = w0;
                rem += UNR * RG;                                   // < 2 * rows_per_example here
                if (rem >= rows_per_example) { rem -= rows_per_example; ++e; }
            } else {
#pragma unroll
                for (int k = 0; k < UNR; ++k) { w[k] = __ldg(clip + e); advance(RG); }
            }
        }
#pragma unroll
        for (int k = 0; k < UNR; ++k) {
            float hf[VEC], zf[VEC];
            ew_f32(h[k], hf); ew_f32(z[k], zf);
#pragma unroll
            for (int u = 0; u < VEC; ++u) {
                const float zw = WEIGHTED ? zf[u] * w[k] : zf[u];
                gg[u] = fmaf(zw, hf[u], gg[u]);
                gs[u] += zw;
            }
        }
    }
    for (; r < r1; r += RG) {
        EwRaw<T, VEC> h, z;
        ew_load(H + (size_t)r * ldh + c0, h);
        ew_load(Z + (size_t)r * ldz + c0, z);
        float w = 1.f;
        if (WEIGHTED) { w = __ldg(clip + e); advance(RG); }
        float hf[VEC], zf[VEC];
        ew_f32(h, hf); ew_f32(z, zf);
#pragma unroll
        for (int u = 0; u < VEC; ++u) {
            const float zw = WEIGHTED ? zf[u] * w : zf[u];
            gg[u] = fmaf(zw, hf[u], gg[u]);
            gs[u] += zw;
        }
    }
}

// Sum the row groups' partial column sums; valid in the threads of row group 0.
template <int VEC, int CG>
__device__ __forceinline__ void ew_combine(float (&gg)[VEC], float (&gs)[VEC], int cg, int rg, float* smem) {
    constexpr int RG = EW_THREADS / CG;
    float* mine = smem + ((rg * CG + cg) * 2) * VEC;
    if (rg > 0) {
#pragma unroll
        for (int u = 0; u < VEC; ++u) { mine[u] = gg[u]; mine[VEC + u] = gs[u]; }
    }
    __syncthreads();
    if (rg == 0) {
#pragma unroll
        for (int g = 1; g < RG; ++g) {
            const float* o = smem + ((g * CG + cg) * 2) * VEC;
#pragma unroll
            for (int u = 0; u < VEC; ++u) { gg[u] += o[u]; gs[u] += o[VEC + u]; }
        }
    }
}

// CG column groups of VEC columns per CTA (CG = 64 or 32: narrower CTAs when the grid would not fill the GPU).
template <typename T, int VEC, int CG>
__global__ void __launch_bounds__(EW_THREADS)
elementwise_norm_kernel(const T* __restrict__ H, long ldh, const T* __restrict__ Z, long ldz, int rows, int d,
                        int has_shift, float* __restrict__ sq, int use_atomic) {
    constexpr int RG = EW_THREADS / CG;
    __shared__ float part[EW_THREADS * 2 * VEC];
    __shared__ float red[32];
    const int cg = threadIdx.x % CG, rg = threadIdx.x / CG;
    const int c0 = (blockIdx.x * CG + cg) * VEC;
    const int i = blockIdx.y;
    float gg[VEC], gs[VEC];
#pragma unroll
    for (int u = 0; u < VEC; ++u) { gg[u] = 0.f; gs[u] = 0.f; }
    if (c0 < d)
        ew_accumulate<T, VEC, RG, false>(H, ldh, Z, ldz, (long)i * rows, (long)(i + 1) * rows, rows, nullptr, c0, rg, gg, gs);
    ew_combine<VEC, CG>(gg, gs, cg, rg, part);
    float s = 0.f;
    if (rg == 0 && c0 < d) {
#pragma unroll
        for (int u = 0; u < VEC; ++u) { s = fmaf(gg[u], gg[u], s); if (has_shift) s = fmaf(gs[u], gs[u], s); }
    }
    s = block_sum(s, red);
    if (threadIdx.x == 0) { if (use_atomic) atomicAdd(sq + i, s); else sq[i] = s; }
}

template <typename T, int VEC, int CG>
__global__ void __launch_bounds__(EW_THREADS)
elementwise_grad_kernel(const T* __restrict__ H, long ldh, const T* __restrict__ Z, long ldz, long rows_total,
                        long rows_per_cta, int rows_per_example, int d, const float* __restrict__ clip,
                        float* __restrict__ g_scale, float* __restrict__ g_shift) {
    constexpr int RG = EW_THREADS / CG;
    __shared__ float part[EW_THREADS * 2 * VEC];
    const int cg = threadIdx.x % CG, rg = threadIdx.x / CG;
    const int c0 = (blockIdx.x * CG + cg) * VEC;
    const long r0 = (long)blockIdx.y * rows_per_cta;
    const long r1 = r0 + rows_per_cta < rows_total ? r0 + rows_per_cta : rows_total;
    float gg[VEC], gs[VEC];
#pragma unroll
    for (int u = 0; u < VEC; ++u) { gg[u] = 0.f; gs[u] = 0.f; }
    if (c0 < d) {
        if (clip) ew_accumulate<T, VEC, RG, true>(H, ldh, Z, ldz, r0, r1, rows_per_example, clip, c0, rg, gg, gs);
        else ew_accumulate<T, VEC, RG, false>(H, ldh, Z, ldz, r0, r1, rows_per_example, nullptr, c0, rg, gg, gs);
    }
    ew_combine<VEC, CG>(gg, gs, cg, rg, part);
    if (rg == 0 && c0 < d) {
#pragma unroll
        for (int u = 0; u < VEC; ++u) {
            atomicAdd(g_scale + c0 + u, gg[u]);
            if (g_shift) atomicAdd(g_shift + c0 + u, gs[u]);
        }
    }
}

// Launch helpers of the element-wise layer kernels: VEC = 4 needs 4-element-aligned rows and width; CG = 32
// (narrower CTAs, more of them) when 64-column-group CTAs would leave SMs idle.
template <typename T>
void launch_ew_norm(bool vec, int cg, dim3 grid, cudaStream_t st, const void* H, long ldh, const void* Z, long ldz,
                    int T_, int d, int has_shift, float* sq, int use_atomic) {
    const T* h = static_cast<const T*>(H); const T* z = static_cast<const T*>(Z);
    if (vec && cg == 64) elementwise_norm_kernel<T, 4, 64><<<grid, EW_THREADS, 0, st>>>(h, ldh, z, ldz, T_, d, has_shift, sq, use_atomic);
    else if (vec) elementwise_norm_kernel<T, 4, 32><<<grid, EW_THREADS, 0, st>>>(h, ldh, z, ldz, T_, d, has_shift, sq, use_atomic);
    else if (cg == 64) elementwise_norm_kernel<T, 1, 64><<<grid, EW_THREADS, 0, st>>>(h, ldh, z, ldz, T_, d, has_shift, sq, use_atomic);
    else elementwise_norm_kernel<T, 1, 32><<<grid, EW_THREADS, 0, st>>>(h, ldh, z, ldz, T_, d, has_shift, sq, use_atomic);
}
template <typename T>
void launch_ew_grad(bool vec, int cg, dim3 grid, cudaStream_t st, const void* H, long ldh, const void* Z, long ldz,
                    long R, long rows_per_cta, int T_, int d, const float* clip, float* g_scale, float* g_shift) {
    const T* h = static_cast<const T*>(H); const T* z = static_cast<const T*>(Z);
    if (vec && cg == 64) elementwise_grad_kernel<T, 4, 64><<<grid, EW_THREADS, 0, st>>>(h, ldh, z, ldz, R, rows_per_cta, T_, d, clip, g_scale, g_shift);
    else if (vec) elementwise_grad_kernel<T, 4, 32><<<grid, EW_THREADS, 0, st>>>(h, ldh, z, ldz, R, rows_per_cta, T_, d, clip, g_scale, g_shift);
    else if (cg == 64) elementwise_grad_kernel<T, 1, 64><<<grid, EW_THREADS, 0, st>>>(h, ldh, z, ldz, R, rows_per_cta, T_, d, clip, g_scale, g_shift);
    else elementwise_grad_kernel<T, 1, 32><<<grid, EW_THREADS, 0, st>>>(h, ldh, z, ldz, R, rows_per_cta, T_, d, clip, g_scale, g_shift);
}

}  // namespace dpclip
