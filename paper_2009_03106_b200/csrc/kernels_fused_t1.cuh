// Two-launch whole step for models whose layers all have T = 1 (dense MLPs).
//
// At these sizes (a few MB of inputs, a few MB of outputs) the step is bound by
// launch latency, not by HBM: one kernel per layer and stage costs more than
// the work.  Here the whole path is two kernels; the kernel boundary is the
// only grid-wide dependency (every example's factor needs all its layers).
//
//   t1_all_norms_kernel : one warp per (layer, example) row pair, closed form
//                         ||a||^2 ||zb||^2 (+ ||zb||^2), writes sq[l][i].
//   t1_all_grads_kernel : every CTA first rebuilds the B clip factors from sq
//                         (L*B floats, L2-resident) into shared memory, then
//                         walks 64 x 64 output tiles of ALL layers; K = B rows,
//                         diag(c) applied as the zb row is loaded, bias as the
//                         extra all-ones column, Philox noise added in the
//                         epilogue, so each output element is written once.
#pragma once
#include "kernels_simt.cuh"
#include "kernels_stream.cuh"

namespace dpclip {

constexpr int FUSED_MAX_LAYERS = 8;
constexpr int FUSED_MAX_B = 2048;

struct FusedT1Layer {
    const void* A; long lda;
    const void* Z; long ldz;
    int d_in, d_out, has_bias;
    int vec_a, vec_z;
    float* gW; float* gb;          // dense rows (ldg == d_in)
    int tiles_m, tiles_n, tile_begin;
};

struct FusedT1Params {
    FusedT1Layer layer[FUSED_MAX_LAYERS];
    int L, B, total_tiles;
    float C, noise_scale;
    uint32_t k0, k1;               // Philox key
    unsigned long long stream_id0;
    float* sq; float* clip; float* norms;
};

template <typename T>
__global__ void __launch_bounds__(128)
t1_all_norms_kernel(const __grid_constant__ FusedT1Params p) {
    const int warp = (blockIdx.x * blockDim.x + threadIdx.x) >> 5, lane = threadIdx.x & 31;
    if (warp >= p.L * p.B) return;
    const int l = warp / p.B, i = warp - l * p.B;
    const FusedT1Layer& y = p.layer[l];
    const T* a = static_cast<const T*>(y.A) + (size_t)i * y.lda;
    const T* z = static_cast<const T*>(y.Z) + (size_t)i * y.ldz;
    float sa = 0.f, sz = 0.f;
    int done = 0;
    if (y.vec_a) {
        for (int j = lane; j < (y.d_in >> 2); j += 32) {
            const float4 v = load4(a + 4 * j);
            sa = fmaf(v.x, v.x, sa); sa = fmaf(v.y, v.y, sa); sa = fmaf(v.z, v.z, sa); sa = fmaf(v.w, v.w, sa);
        }
        done = y.d_in & ~3;
    }
    for (int j = done + lane; j < y.d_in; j += 32) { const float v = to_f32(a[j]); sa = fmaf(v, v, sa); }
    done = 0;
    if (y.vec_z) {
        for (int j = lane; j < (y.d_out >> 2); j += 32) {
            const float4 v = load4(z + 4 * j);
            sz = fmaf(v.x, v.x, sz); sz = fmaf(v.y, v.y, sz); sz = fmaf(v.z, v.z, sz); sz = fmaf(v.w, v.w, sz);
        }
        done = y.d_out & ~3;
    }
    for (int j = done + lane; j < y.d_out; j += 32) { const float v = to_f32(z[j]); sz = fmaf(v, v, sz); }
    sa = warp_sum(sa);
    sz = warp_sum(sz);
    if (lane == 0) p.sq[(size_t)l * p.B + i] = (sa + (y.has_bias ? 1.f : 0.f)) * sz;
}

template <typename T>
__global__ void __launch_bounds__(SIMT_THREADS)
t1_all_grads_kernel(const __grid_constant__ FusedT1Params p) {
    __shared__ __align__(16) float Zs[2][SIMT_BK][SIMT_BM];
    __shared__ __align__(16) float As[2][SIMT_BK][SIMT_BN];
    __shared__ float clip_s[FUSED_MAX_B];

    const int tid = threadIdx.x;
    // factors, rebuilt by every CTA (cheaper than a third launch or a grid barrier)
    for (int i = tid; i < p.B; i += SIMT_THREADS) {
        float s = 0.f;
        for (int l = 0; l < p.L; ++l) s += p.sq[(size_t)l * p.B + i];
        const float n = sqrtf(s);
        const float c = n > p.C ? p.C / n : 1.0f;
        clip_s[i] = c;
        if (blockIdx.x == 0) { p.clip[i] = c; if (p.norms) p.norms[i] = n; }
    }
    __syncthreads();

    const int ty = tid >> 4, tx = tid & 15;
    const int lk = tid >> 4, lc = (tid & 15) << 2;
    const int n_slabs = (p.B + SIMT_BK - 1) / SIMT_BK;

    for (int tile = blockIdx.x; tile < p.total_tiles; tile += gridDim.x) {
        int l = 0;
        while (l + 1 < p.L && tile >= p.layer[l + 1].tile_begin) ++l;
        const FusedT1Layer& y = p.layer[l];
        const int local = tile - y.tile_begin;
        const int m0 = (local / y.tiles_n) * SIMT_BM, n0 = (local % y.tiles_n) * SIMT_BN;
        const T* __restrict__ A = static_cast<const T*>(y.A);
        const T* __restrict__ Z = static_cast<const T*>(y.Z);

        float acc[4][4];
#pragma unroll
        for (int i = 0; i < 4; ++i)
#pragma unroll
            for (int j = 0; j < 4; ++j) acc[i][j] = 0.f;

        auto fetch = [&](int slab, float4& zr, float4& ar) {
            const int r = slab * SIMT_BK + lk;
            const bool ok = r < p.B;
            zr = simt_load_row4(Z, y.ldz, r, m0 + lc, y.d_out, ok, y.vec_z != 0, false);
            ar = simt_load_row4(A, y.lda, r, n0 + lc, y.d_in, ok, y.vec_a != 0, y.has_bias != 0);
            if (ok) { const float c = clip_s[r]; zr.x *= c; zr.y *= c; zr.z *= c; zr.w *= c; }
        };
        float4 zr, ar;
        fetch(0, zr, ar);
        __syncthreads();                                   // previous tile's readers are done with buffer 0
        *reinterpret_cast<float4*>(&Zs[0][lk][lc]) = zr;
        *reinterpret_cast<float4*>(&As[0][lk][lc]) = ar;
        __syncthreads();
        for (int s = 0; s < n_slabs; ++s) {
            const int buf = s & 1;
            const bool more = s + 1 < n_slabs;
            if (more) fetch(s + 1, zr, ar);
#pragma unroll
            for (int k = 0; k < SIMT_BK; ++k) {
                const float4 zv = *reinterpret_cast<const float4*>(&Zs[buf][k][ty << 2]);
                const float4 av = *reinterpret_cast<const float4*>(&As[buf][k][tx << 2]);
                const float zz[4] = {zv.x, zv.y, zv.z, zv.w};
                const float aa[4] = {av.x, av.y, av.z, av.w};
#pragma unroll
                for (int i = 0; i < 4; ++i)
#pragma unroll
                    for (int j = 0; j < 4; ++j) acc[i][j] = fmaf(zz[i], aa[j], acc[i][j]);
            }
            if (more) {
                *reinterpret_cast<float4*>(&Zs[buf ^ 1][lk][lc]) = zr;
                *reinterpret_cast<float4*>(&As[buf ^ 1][lk][lc]) = ar;
            }
            __syncthreads();
        }

        // epilogue: + noise, single store per element
        const unsigned long long sid_w = p.stream_id0 + 2ull * l, sid_b = sid_w + 1;
        const int n = n0 + (tx << 2);
#pragma unroll
        for (int i = 0; i < 4; ++i) {
            const int m = m0 + (ty << 2) + i;
            if (m >= y.d_out) continue;
            float out[4] = {acc[i][0], acc[i][1], acc[i][2], acc[i][3]};
            if (p.noise_scale > 0.f) {
                const size_t j0 = (size_t)m * y.d_in + n;
                if ((y.d_in & 3) == 0 && n + 4 <= y.d_in) {        // the four columns are one Philox block
                    const size_t q = j0 >> 2;
                    PhiloxBlock b = philox_block((uint32_t)q, (uint32_t)(q >> 32), (uint32_t)sid_w,
                                                 (uint32_t)(sid_w >> 32), p.k0, p.k1);
                    float z4[4];
                    box_muller(b.v[0], b.v[1], z4[0], z4[1]);
                    box_muller(b.v[2], b.v[3], z4[2], z4[3]);
#pragma unroll
                    for (int j = 0; j < 4; ++j) out[j] = fmaf(p.noise_scale, z4[j], out[j]);
                } else {
#pragma unroll
                    for (int j = 0; j < 4; ++j) {
                        const int nn = n + j;
                        if (nn > y.d_in || (nn == y.d_in && !y.has_bias)) continue;
                        const bool is_bias = nn == y.d_in;
                        const size_t e = is_bias ? (size_t)m : j0 + j;
                        const unsigned long long sid = is_bias ? sid_b : sid_w;
                        const size_t q = e >> 2;
                        PhiloxBlock b = philox_block((uint32_t)q, (uint32_t)(q >> 32), (uint32_t)sid,
                                                     (uint32_t)(sid >> 32), p.k0, p.k1);
                        float za, zb;
                        box_muller(b.v[(e & 2)], b.v[(e & 2) + 1], za, zb);
                        out[j] = fmaf(p.noise_scale, (e & 1) ? zb : za, out[j]);
                    }
                }
            }
            float* row = y.gW + (size_t)m * y.d_in;
            if (n + 4 <= y.d_in && (y.d_in & 3) == 0) {
                *reinterpret_cast<float4*>(row + n) = make_float4(out[0], out[1], out[2], out[3]);
            } else {
#pragma unroll
                for (int j = 0; j < 4; ++j) {
                    const int nn = n + j;
                    if (nn < y.d_in) row[nn] = out[j];
                    else if (nn == y.d_in && y.has_bias && y.gb) y.gb[m] = out[j];
                }
            }
        }
    }
}

}  // namespace dpclip
