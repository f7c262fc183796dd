// Bandwidth-bound streaming kernels: T=1 squared norms, clip factors, noise.
#pragma once
#include "common.cuh"

namespace dpclip {

// ---------------------------------------------------------------------------
// T = 1 layer norms (Goodfellow's closed form): the per-example gradient is
// the outer product zb (x) a, so ||G||_F^2 = ||zb||^2 ||a||^2, and the bias
// gradient is zb itself, so with a bias the total is (||a||^2 + 1) ||zb||^2.
// Each row of A and Zbar is read exactly once with 128-bit (fp32) / 64-bit
// (bf16) loads when aligned; one CTA per example, shuffle + smem reduction.
// ---------------------------------------------------------------------------
template <typename T>
__device__ __forceinline__ float row_sumsq(const T* __restrict__ row, int n, bool vec_ok) {
    float s0 = 0.f, s1 = 0.f, s2 = 0.f, s3 = 0.f;
    int done = 0;
    if (vec_ok) {
        int nv = n >> 2;
        for (int j = threadIdx.x; j < nv; j += blockDim.x) {
            float4 v = load4(row + 4 * j);
            s0 = fmaf(v.x, v.x, s0); s1 = fmaf(v.y, v.y, s1);
            s2 = fmaf(v.z, v.z, s2); s3 = fmaf(v.w, v.w, s3);
        }
        done = nv << 2;
    }
    for (int j = done + threadIdx.x; j < n; j += blockDim.x) {
        float v = to_f32(row[j]);
        s0 = fmaf(v, v, s0);
    }
    return (s0 + s1) + (s2 + s3);
}

template <typename T>
__global__ void __launch_bounds__(256)
t1_sqnorm_kernel(const T* __restrict__ A, long lda, const T* __restrict__ Z, long ldz,
                 int d_in, int d_out, int has_bias, int vec_a, int vec_z, float* __restrict__ sq) {
    __shared__ float red[32];
    const int i = blockIdx.x;
    float sa = row_sumsq(A + (size_t)i * lda, d_in, vec_a != 0);
    float sz = row_sumsq(Z + (size_t)i * ldz, d_out, vec_z != 0);
    sa = block_sum(sa, red);
    sz = block_sum(sz, red);
    if (threadIdx.x == 0) sq[i] = (sa + (has_bias ? 1.f : 0.f)) * sz;
}

// ---------------------------------------------------------------------------
// Cross-layer accumulate + clip factors.  One CTA; B is at most a few
// thousand, the kernel is pure latency.
// ---------------------------------------------------------------------------
__global__ void __launch_bounds__(256)
factors_kernel(const float* __restrict__ sq_layers, int L, long ld_sq, int B, float C,
               float* __restrict__ clip, float* __restrict__ norms, int* __restrict__ n_clipped) {
    __shared__ float red[32];
    float cnt = 0.f;
    for (int i = threadIdx.x; i < B; i += blockDim.x) {
        float s = 0.f;
        for (int l = 0; l < L; ++l) s += sq_layers[(size_t)l * ld_sq + i];
        float n = sqrtf(s);
        float c = 1.0f;
        if (n > C) { c = C / n; cnt += 1.f; }       // tie and zero norm stay exactly 1
        clip[i] = c;
        if (norms) norms[i] = n;
    }
    if (n_clipped) {
        cnt = block_sum(cnt, red);
        if (threadIdx.x == 0) n_clipped[0] = (int)cnt;
    }
}

// Per-layer clipping (Sec. "Related Work"): row l of sq[L][B] gives layer l's own factors against its own
// threshold C[l].  One CTA per layer.
struct LayerThresholds { float C[64]; };
__global__ void __launch_bounds__(256)
factors_rows_kernel(const float* __restrict__ sq_layers, long ld_sq, int B, const LayerThresholds th,
                    float* __restrict__ clip_layers, float* __restrict__ norms_layers) {
    const int l = blockIdx.x;
    const float C = th.C[l];
    for (int i = threadIdx.x; i < B; i += blockDim.x) {
        const float n = sqrtf(sq_layers[(size_t)l * ld_sq + i]);
        float c = 1.0f;
        if (n > C) c = C / n;                         // tie and zero norm stay exactly 1
        clip_layers[(size_t)l * B + i] = c;
        if (norms_layers) norms_layers[(size_t)l * B + i] = n;
    }
}

// ---------------------------------------------------------------------------
// Gaussian noise: Philox4x32-10 counter-based generator + Box-Muller.
// One 128-bit block gives four normals; a thread owns block q = elements
// 4q..4q+3, so the output depends only on (seed, stream_id, element index).
// ---------------------------------------------------------------------------
struct PhiloxBlock { uint32_t v[4]; };

__device__ __forceinline__ PhiloxBlock philox_block(uint32_t c0, uint32_t c1, uint32_t c2, uint32_t c3,
                                                    uint32_t k0, uint32_t k1) {
#pragma unroll
    for (int r = 0; r < 10; ++r) {
        const uint32_t hi0 = __umulhi(0xD2511F53u, c0), lo0 = 0xD2511F53u * c0;
        const uint32_t hi1 = __umulhi(0xCD9E8D57u, c2), lo1 = 0xCD9E8D57u * c2;
        c0 = hi1 ^ c1 ^ k0;
        c1 = lo1;
        c2 = hi0 ^ c3 ^ k1;
        c3 = lo0;
        k0 += 0x9E3779B9u;
        k1 += 0xBB67AE85u;
    }
    PhiloxBlock b;
    b.v[0] = c0; b.v[1] = c1; b.v[2] = c2; b.v[3] = c3;
    return b;
}

__device__ __forceinline__ float bits_to_u01(uint32_t x) {          // (0, 1]
    return __fmaf_rn(__uint2float_rn(x), 2.3283064365386963e-10f, 1.1641532182693481e-10f);
}

// Box-Muller pair from two 32-bit draws.  The generator costs more issue slots than anything else in the
// small fused steps, so it uses the hardware approximations where their error stays well inside the
// 1e-5 absolute budget of a standard normal (every kernel shares this one function, so all launch
// forms give the same bits):
//   ln u1 : lg2.approx (relative error 2^-22 below 1/2, absolute 2^-22 above); within 2^-7 of 1, where an
//           absolute error would dominate the small radius, the series -w - w^2/2 - w^3/3 - w^4/4, w = 1 - u1
//   sqrt  : sqrt.approx (about 1 ulp)
//   angle : 2 pi (u2 - 1/2) lies in (-pi, pi], where sin/cos.approx are good to 2^-20.9 absolute;
//           cos(2 pi u2) = -cos(2 pi (u2 - 1/2)), likewise for sin
__device__ __forceinline__ void box_muller(uint32_t xa, uint32_t xb, float& n0, float& n1) {
    const float u1 = bits_to_u01(xa), u2 = bits_to_u01(xb);
    float l2;
    asm("lg2.approx.ftz.f32 %0, %1;" : "=f"(l2) : "f"(u1));
    const float w = 1.0f - u1;                                  // exact for u1 >= 1/2
    const float series = -w * fmaf(w, fmaf(w, fmaf(w, 0.25f, 0.333333343f), 0.5f), 1.0f);
    const float ln = w < 0.0078125f ? series : l2 * 0.693147182f;
    float r;
    asm("sqrt.approx.ftz.f32 %0, %1;" : "=f"(r) : "f"(-2.0f * ln));
    const float th = 6.28318548f * (u2 - 0.5f);
    float s, c;
    asm("sin.approx.ftz.f32 %0, %1;" : "=f"(s) : "f"(th));
    asm("cos.approx.ftz.f32 %0, %1;" : "=f"(c) : "f"(th));
    n0 = -r * c;
    n1 = -r * s;
}

__global__ void __launch_bounds__(256)
noise_kernel(float* __restrict__ g, size_t n, float scale, uint32_t k0, uint32_t k1,
             uint32_t s0, uint32_t s1, int vec_ok) {
    const size_t nq = (n + 3) >> 2;
    const size_t stride = (size_t)gridDim.x * blockDim.x;
    for (size_t q = (size_t)blockIdx.x * blockDim.x + threadIdx.x; q < nq; q += stride) {
        PhiloxBlock b = philox_block((uint32_t)q, (uint32_t)(q >> 32), s0, s1, k0, k1);
        float z[4];
        box_muller(b.v[0], b.v[1], z[0], z[1]);
        box_muller(b.v[2], b.v[3], z[2], z[3]);
        const size_t j = q << 2;
        if (vec_ok && j + 3 < n) {
            float4 v = *reinterpret_cast<float4*>(g + j);
            v.x = fmaf(scale, z[0], v.x); v.y = fmaf(scale, z[1], v.y);
            v.z = fmaf(scale, z[2], v.z); v.w = fmaf(scale, z[3], v.w);
            *reinterpret_cast<float4*>(g + j) = v;
        } else {
#pragma unroll
            for (int e = 0; e < 4; ++e)
                if (j + e < n) g[j + e] = fmaf(scale, z[e], g[j + e]);
        }
    }
}

// ---------------------------------------------------------------------------
// Parameter updates with the noise folded in (one pass over the parameters instead of a noise pass
// followed by an optimiser pass).  g = (gsum + scale * xi) * inv_tau is the noisy mean gradient of
// Algorithm 1's last line; ADAM = false applies theta -= lr * g, ADAM = true the Adam rule with bias
// corrections c1 = 1 - beta1^t, c2 = 1 - beta2^t computed on the host.
// ---------------------------------------------------------------------------
struct UpdateParams {
    float* theta; float* m; float* v; const float* gsum; size_t n;
    float inv_tau, scale, lr, beta1, beta2, eps, inv_c1, inv_c2;
    uint32_t k0, k1, s0, s1;
    int vec_ok;
};

template <bool ADAM>
__global__ void __launch_bounds__(256)
dp_update_kernel(const UpdateParams p) {
    const size_t nq = (p.n + 3) >> 2;
    const size_t stride = (size_t)gridDim.x * blockDim.x;
    for (size_t q = (size_t)blockIdx.x * blockDim.x + threadIdx.x; q < nq; q += stride) {
        const size_t j = q << 2;
        const bool full = p.vec_ok && j + 3 < p.n;
        float g[4], th[4], mm[4], vv[4];
        if (full) {
            const float4 a = *reinterpret_cast<const float4*>(p.gsum + j), b = *reinterpret_cast<const float4*>(p.theta + j);
            g[0] = a.x; g[1] = a.y; g[2] = a.z; g[3] = a.w; th[0] = b.x; th[1] = b.y; th[2] = b.z; th[3] = b.w;
            if (ADAM) {
                const float4 c = *reinterpret_cast<const float4*>(p.m + j), d = *reinterpret_cast<const float4*>(p.v + j);
                mm[0] = c.x; mm[1] = c.y; mm[2] = c.z; mm[3] = c.w; vv[0] = d.x; vv[1] = d.y; vv[2] = d.z; vv[3] = d.w;
            }
        } else {
#pragma unroll
            for (int e = 0; e < 4; ++e) {
                const bool in = j + e < p.n;
                g[e] = in ? p.gsum[j + e] : 0.f; th[e] = in ? p.theta[j + e] : 0.f;
                if (ADAM) { mm[e] = in ? p.m[j + e] : 0.f; vv[e] = in ? p.v[j + e] : 0.f; }
            }
        }
        float z[4] = {0.f, 0.f, 0.f, 0.f};
        if (p.scale > 0.f) {
            PhiloxBlock b = philox_block((uint32_t)q, (uint32_t)(q >> 32), p.s0, p.s1, p.k0, p.k1);
            box_muller(b.v[0], b.v[1], z[0], z[1]);
            box_muller(b.v[2], b.v[3], z[2], z[3]);
        }
#pragma unroll
        for (int e = 0; e < 4; ++e) {
            const float gn = fmaf(p.scale, z[e], g[e]) * p.inv_tau;
            if (ADAM) {
                mm[e] = fmaf(p.beta1, mm[e], (1.f - p.beta1) * gn);
                vv[e] = fmaf(p.beta2, vv[e], (1.f - p.beta2) * gn * gn);
                th[e] -= p.lr * (mm[e] * p.inv_c1) / (sqrtf(vv[e] * p.inv_c2) + p.eps);
            } else {
                th[e] = fmaf(-p.lr, gn, th[e]);
            }
        }
        if (full) {
            *reinterpret_cast<float4*>(p.theta + j) = make_float4(th[0], th[1], th[2], th[3]);
            if (ADAM) {
                *reinterpret_cast<float4*>(p.m + j) = make_float4(mm[0], mm[1], mm[2], mm[3]);
                *reinterpret_cast<float4*>(p.v + j) = make_float4(vv[0], vv[1], vv[2], vv[3]);
            }
        } else {
#pragma unroll
            for (int e = 0; e < 4; ++e)
                if (j + e < p.n) { p.theta[j + e] = th[e]; if (ADAM) { p.m[j + e] = mm[e]; p.v[j + e] = vv[e]; } }
        }
    }
}

// Noise on every released tensor of a model in ONE launch (the weights and the bias of layer l are
// tensors 2l and 2l + 1, with their own noise streams).  Blocks are dealt to tensors by a prefix table.
constexpr int NOISE_BATCH_MAX = 128;
struct NoiseBatchParams {
    float* g[NOISE_BATCH_MAX];
    unsigned long long n[NOISE_BATCH_MAX];
    unsigned long long sid[NOISE_BATCH_MAX];
    int blk_begin[NOISE_BATCH_MAX + 1];          // first block of tensor k; blk_begin[count] = grid size
    int count;
    float scale; uint32_t k0, k1;
};

__global__ void __launch_bounds__(256)
noise_batch_kernel(const __grid_constant__ NoiseBatchParams p) {
    int k = 0;
    while (k + 1 < p.count && (int)blockIdx.x >= p.blk_begin[k + 1]) ++k;
    float* __restrict__ g = p.g[k];
    const size_t n = p.n[k], nq = (n + 3) >> 2;
    const uint32_t s0 = (uint32_t)p.sid[k], s1 = (uint32_t)(p.sid[k] >> 32);
    const bool vec_ok = (reinterpret_cast<uintptr_t>(g) & 15) == 0;
    const size_t stride = (size_t)(p.blk_begin[k + 1] - p.blk_begin[k]) * blockDim.x;
    for (size_t q = (size_t)(blockIdx.x - p.blk_begin[k]) * blockDim.x + threadIdx.x; q < nq; q += stride) {
        PhiloxBlock b = philox_block((uint32_t)q, (uint32_t)(q >> 32), s0, s1, p.k0, p.k1);
        float z[4];
        box_muller(b.v[0], b.v[1], z[0], z[1]);
        box_muller(b.v[2], b.v[3], z[2], z[3]);
        const size_t j = q << 2;
        if (vec_ok && j + 3 < n) {
            float4 v = *reinterpret_cast<float4*>(g + j);
            v.x = fmaf(p.scale, z[0], v.x); v.y = fmaf(p.scale, z[1], v.y);
            v.z = fmaf(p.scale, z[2], v.z); v.w = fmaf(p.scale, z[3], v.w);
            *reinterpret_cast<float4*>(g + j) = v;
        } else {
#pragma unroll
            for (int e = 0; e < 4; ++e)
                if (j + e < n) g[j + e] = fmaf(p.scale, z[e], g[j + e]);
        }
    }
}

// Patch matrix of a convolution written out, [B*T][C*kh*kw] fp32 with columns in (c, ky, kx) order and zeros
// for the padding (Sec. "Convolutional Layers": the unfolded input).  Only for first layers whose patch rows are
// at most 32 columns: there the packed narrow tensor-core kernel on the patch matrix beats the implicit forms,
// and the matrix is a few MB.  CTA = 64 rows; lane = patch column (its (c, ky, kx) worked out once), warp w takes
// rows w, w + 8, ...: a warp writes one row's d_in consecutive floats, rows back to back.
__global__ void __launch_bounds__(256)
im2col_f32_kernel(const float* __restrict__ X, float* __restrict__ P, int rows, int T, int d_in, int C, int H, int W,
                  int kh, int kw, int stride, int pad, int Wo) {
    const int n = threadIdx.x & 31, w = threadIdx.x >> 5;
    if (n >= d_in) return;
    const int c = n / (kh * kw), r = n - c * kh * kw, ky = r / kw, kx = r - ky * kw;
    const int row0 = blockIdx.x * 64;
#pragma unroll 4
    for (int i = 0; i < 8; ++i) {
        const int row = row0 + w + 8 * i;
        if (row >= rows) break;
        const int b = row / T, t = row - b * T;
        const int yo = t / Wo, xo = t - yo * Wo;
        const int y = yo * stride - pad + ky, x = xo * stride - pad + kx;
        float v = 0.f;
        if (y >= 0 && y < H && x >= 0 && x < W) v = __ldg(X + (((size_t)b * C + c) * H + y) * W + x);
        P[(size_t)row * d_in + n] = v;
    }
}

// dL/dZ of a convolution as a framework holds it, [B][d_out][T] (channel-major), rewritten as [B][T][d_out]
// for the kernels that read [row][feature] tiles: 32 x 32 tiles through shared memory, reads and writes
// both 128-byte coalesced.  grid = (ceil(T / 32), ceil(d_out / 32), B), 256 threads.
__global__ void __launch_bounds__(256)
channel_major_to_rows_kernel(const float* __restrict__ src, float* __restrict__ dst, int d_out, int T) {
    __shared__ float tile[32][33];
    const size_t base = (size_t)blockIdx.z * d_out * T;
    const int t0 = blockIdx.x * 32, m0 = blockIdx.y * 32;
    const int tx = threadIdx.x & 31, ty = threadIdx.x >> 5;
#pragma unroll
    for (int i = 0; i < 4; ++i) {
        const int m = m0 + ty + 8 * i, t = t0 + tx;
        if (m < d_out && t < T) tile[ty + 8 * i][tx] = src[base + (size_t)m * T + t];
    }
    __syncthreads();
#pragma unroll
    for (int i = 0; i < 4; ++i) {
        const int t = t0 + ty + 8 * i, m = m0 + tx;
        if (t < T && m < d_out) dst[base + (size_t)t * d_out + m] = tile[tx][ty + 8 * i];
    }
}

}  // namespace dpclip
