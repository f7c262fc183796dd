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
    int index;                     // position of the layer in the caller's model: row of sq, noise stream ids
};

struct FusedT1Params {
    FusedT1Layer layer[FUSED_MAX_LAYERS];
    int L, B, total_tiles;
    float C, noise_scale;
    uint32_t k0, k1;               // Philox key
    unsigned long long stream_id0;
    float* sq; float* clip; float* norms;
    const float* clip_in;          // factors already known (T = 1 layers of a mixed model): sq is not summed
};

// one CTA of 128 threads per (layer, example): every thread has at most a few independent 128-bit
// loads, all in flight at once (the kernel is pure memory latency)
template <typename T>
__global__ void __launch_bounds__(128)
t1_all_norms_kernel(const __grid_constant__ FusedT1Params p) {
    __shared__ float red[32];
    const int l = blockIdx.x / p.B, i = blockIdx.x - l * p.B;
    const FusedT1Layer& y = p.layer[l];
    const T* a = static_cast<const T*>(y.A) + (size_t)i * y.lda;
    const T* z = static_cast<const T*>(y.Z) + (size_t)i * y.ldz;
    float sa = row_sumsq(a, y.d_in, y.vec_a != 0);
    float sz = row_sumsq(z, y.d_out, y.vec_z != 0);
    sa = block_sum(sa, red);
    sz = block_sum(sz, red);
    if (threadIdx.x == 0) p.sq[(size_t)y.index * p.B + i] = (sa + (y.has_bias ? 1.f : 0.f)) * sz;
}

// One row of four consecutive outputs (m, n .. n+3) of layer y: add the noise, store once.
// Column d_in of the tile is the bias gradient (the all-ones column of [A | 1]).
__device__ __forceinline__ void fused_t1_emit4(const FusedT1Params& p, const FusedT1Layer& y, int l, int m, int n,
                                               float (&out)[4]) {
    if (m >= y.d_out || n > y.d_in) return;
    const unsigned long long sid_w = p.stream_id0 + 2ull * y.index, sid_b = sid_w + 1;
    const bool row4 = (y.d_in & 3) == 0 && n + 4 <= y.d_in;       // four in-range columns = one Philox block
    if (p.noise_scale > 0.f) {
        const size_t j0 = (size_t)m * y.d_in + n;
        if (row4) {
            const size_t q = j0 >> 2;
            PhiloxBlock b = philox_block((uint32_t)q, (uint32_t)(q >> 32), (uint32_t)sid_w, (uint32_t)(sid_w >> 32),
                                         p.k0, p.k1);
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
                PhiloxBlock b = philox_block((uint32_t)q, (uint32_t)(q >> 32), (uint32_t)sid, (uint32_t)(sid >> 32),
                                             p.k0, p.k1);
                float za, zb;
                box_muller(b.v[(e & 2)], b.v[(e & 2) + 1], za, zb);
                out[j] = fmaf(p.noise_scale, (e & 1) ? zb : za, out[j]);
            }
        }
    }
    float* row = y.gW + (size_t)m * y.d_in;
    if (row4) {
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

// TILE = 64: 4 x 4 outputs per thread, 16-row slabs (small layers; many CTAs hide the load latency).
// TILE = 128: 8 x 8 outputs per thread as 2 x 2 blocks of 4 x 4 (twice the FMAs per shared-memory
//             load), 32-row slabs: one CTA per SM, so each slab issues four 128-bit loads per operand
//             and thread before it waits, and the next slab is in flight during 2048 FMAs per thread.
template <int TILE> struct FusedT1Cfg {
    static constexpr int BK = TILE == 64 ? 16 : 32;
    static constexpr int NL = TILE * BK / 1024;            // float4 loads per thread, operand and slab
    static constexpr int RS = 1024 / TILE;                 // slab rows covered by one pass of the CTA
    static constexpr int SMEM_BYTES = 2 * 2 * BK * TILE * 4 + FUSED_MAX_B * 4;
};

template <typename T, int TILE>
__global__ void __launch_bounds__(SIMT_THREADS)
t1_all_grads_kernel(const __grid_constant__ FusedT1Params p) {
    constexpr int SUB = TILE / 64;
    constexpr int BK = FusedT1Cfg<TILE>::BK, NL = FusedT1Cfg<TILE>::NL, RS = FusedT1Cfg<TILE>::RS;
    extern __shared__ __align__(16) float fused_smem[];
    float (*Zs)[BK][TILE] = reinterpret_cast<float (*)[BK][TILE]>(fused_smem);
    float (*As)[BK][TILE] = reinterpret_cast<float (*)[BK][TILE]>(fused_smem + 2 * BK * TILE);
    float* clip_s = fused_smem + 4 * BK * TILE;

    const int tid = threadIdx.x;
    // factors, rebuilt by every CTA (cheaper than a third launch or a grid barrier)
    for (int i = tid; i < p.B; i += SIMT_THREADS) {
        if (p.clip_in) { clip_s[i] = p.clip_in[i]; continue; }
        float s = 0.f;
        for (int l = 0; l < p.L; ++l) s += p.sq[(size_t)l * p.B + i];
        const float n = sqrtf(s);
        const float c = n > p.C ? p.C / n : 1.0f;
        clip_s[i] = c;
        if (blockIdx.x == 0) { p.clip[i] = c; if (p.norms) p.norms[i] = n; }
    }
    __syncthreads();

    const int ty = tid >> 4, tx = tid & 15;
    const int lk = tid / (TILE / 4), lc = (tid % (TILE / 4)) << 2;
    const int n_slabs = (p.B + BK - 1) / BK;

    for (int tile = blockIdx.x; tile < p.total_tiles; tile += gridDim.x) {
        int l = 0;
        while (l + 1 < p.L && tile >= p.layer[l + 1].tile_begin) ++l;
        const FusedT1Layer& y = p.layer[l];
        const int local = tile - y.tile_begin;
        const int m0 = (local / y.tiles_n) * TILE, n0 = (local % y.tiles_n) * TILE;
        const T* __restrict__ A = static_cast<const T*>(y.A);
        const T* __restrict__ Z = static_cast<const T*>(y.Z);

        float acc[SUB][SUB][4][4];
#pragma unroll
        for (int a = 0; a < SUB; ++a)
#pragma unroll
            for (int b = 0; b < SUB; ++b)
#pragma unroll
                for (int i = 0; i < 4; ++i)
#pragma unroll
                    for (int j = 0; j < 4; ++j) acc[a][b][i][j] = 0.f;

        // fetch() only issues the global loads; the loaded values are first touched in stash(), after
        // the FMAs of the current slab, so the load latency is covered by that work
        float4 zr[NL], ar[NL];
        auto fetch = [&](int slab) {
#pragma unroll
            for (int u = 0; u < NL; ++u) {
                const int r = slab * BK + u * RS + lk;
                const bool ok = r < p.B;
                zr[u] = simt_load_row4(Z, y.ldz, r, m0 + lc, y.d_out, ok, y.vec_z != 0, false);
                ar[u] = simt_load_row4(A, y.lda, r, n0 + lc, y.d_in, ok, y.vec_a != 0, y.has_bias != 0);
            }
        };
        auto stash = [&](int slab, int buf) {
#pragma unroll
            for (int u = 0; u < NL; ++u) {
                const int r = slab * BK + u * RS + lk;
                const float c = r < p.B ? clip_s[r] : 0.f;           // diag(c) on the zb row
                *reinterpret_cast<float4*>(&Zs[buf][u * RS + lk][lc]) =
                    make_float4(zr[u].x * c, zr[u].y * c, zr[u].z * c, zr[u].w * c);
                *reinterpret_cast<float4*>(&As[buf][u * RS + lk][lc]) = ar[u];
            }
        };
        fetch(0);
        __syncthreads();                                   // previous tile's readers are done with buffer 0
        stash(0, 0);
        __syncthreads();
        for (int s = 0; s < n_slabs; ++s) {
            const int buf = s & 1;
            const bool more = s + 1 < n_slabs;
            if (more) fetch(s + 1);
#pragma unroll 8
            for (int k = 0; k < BK; ++k) {
                float zz[SUB][4], aa[SUB][4];
#pragma unroll
                for (int a = 0; a < SUB; ++a) {
                    const float4 zv = *reinterpret_cast<const float4*>(&Zs[buf][k][a * 64 + (ty << 2)]);
                    const float4 av = *reinterpret_cast<const float4*>(&As[buf][k][a * 64 + (tx << 2)]);
                    zz[a][0] = zv.x; zz[a][1] = zv.y; zz[a][2] = zv.z; zz[a][3] = zv.w;
                    aa[a][0] = av.x; aa[a][1] = av.y; aa[a][2] = av.z; aa[a][3] = av.w;
                }
#pragma unroll
                for (int a = 0; a < SUB; ++a)
#pragma unroll
                    for (int b = 0; b < SUB; ++b)
#pragma unroll
                        for (int i = 0; i < 4; ++i)
#pragma unroll
                            for (int j = 0; j < 4; ++j) acc[a][b][i][j] = fmaf(zz[a][i], aa[b][j], acc[a][b][i][j]);
            }
            if (more) stash(s + 1, buf ^ 1);
            __syncthreads();
        }

        // epilogue: + noise, single store per element
#pragma unroll
        for (int a = 0; a < SUB; ++a)
#pragma unroll
            for (int i = 0; i < 4; ++i)
#pragma unroll
                for (int b = 0; b < SUB; ++b)
                    fused_t1_emit4(p, y, l, m0 + a * 64 + (ty << 2) + i, n0 + b * 64 + (tx << 2), acc[a][b][i]);
    }
}

}  // namespace dpclip
