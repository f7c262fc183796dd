// fp32-ALU tile kernel for the product Zbar^T A over a range of rows.
//
// Used (1) for every fp32 layer with T > 1 -- the 1e-5 tolerance of fp32
// inputs rules out plain bf16/tf32 tensor-core math -- and (2) as the path for
// bf16 layers whose rows are not 16-byte multiples (e.g. d_in = 27) and so
// cannot be fetched by TMA.
//
// One CTA computes 64 x 64 output tiles (d_out x d_in) with 4 x 4 register
// micro-tiles, marching over rows in slabs of 16 staged through shared memory
// (register prefetch of the next slab, two smem buffers, one barrier per slab).
// Both operands are read in their native [row][feature] layout, so global
// loads are coalesced along the feature dimension and no transpose is needed.
//
// The bias gradient rides along as one extra column: A is treated as [A | 1],
// so column d_in of the product is sum_t zb_t, the per-example bias gradient.
//
//   NORM mode: rows = the T rows of example blockIdx.y; the tile is squared and
//              summed in registers (Frobenius epilogue); nothing but one float
//              per example leaves the CTA.
//   GRAD mode: rows = one slice of all B*T rows; each Zbar row is multiplied by
//              its example's clip factor as it is loaded (diag(c) fused into
//              the operand load); tiles are stored, or added atomically when
//              the rows are split over several CTAs.
#pragma once
#include "common.cuh"

namespace dpclip {

constexpr int SIMT_BM = 64, SIMT_BN = 64, SIMT_BK = 16, SIMT_THREADS = 256;

struct SimtParams {
    const void* A; long lda;
    const void* Z; long ldz;
    int T, d_in, d_out, has_bias;
    int tiles_m, tiles_n;
    int vec_a, vec_z;              // 4-element vector loads allowed
    // NORM
    float* sq; int use_atomic;
    // GRAD
    const float* clip; float* gW; long ldg; float* gb;
    long rows_total; long rows_per_split;
    // CONV (implicit im2col): A is the feature map [B][C][H][W]; row (i, y', x') and column (c, ky, kx) of the
    // patch matrix are gathered on the fly; Z may be channel-major [B][d_out][T]
    int cC, cH, cW, kh, kw, stride, pad, Wo, z_cm;
};

template <typename T>
__device__ __forceinline__ float4 simt_load_row4(const T* __restrict__ base, long ld, long row, int col,
                                                 int ncols, bool row_ok, bool vec_ok, bool aug) {
    float4 v = make_float4(0.f, 0.f, 0.f, 0.f);
    if (!row_ok) return v;
    const T* p = base + (size_t)row * ld + col;
    if (vec_ok && col + 3 < ncols) return load4(p);
    float e[4];
#pragma unroll
    for (int j = 0; j < 4; ++j) {
        int c = col + j;
        e[j] = c < ncols ? to_f32(p[j]) : ((aug && c == ncols) ? 1.f : 0.f);
    }
    return make_float4(e[0], e[1], e[2], e[3]);
}

// CONV = true: the layer is a convolution given by its INPUT feature map (Algorithm 3 builds the patch
// matrix with unfold; here element (row (i, t), column (c, ky, kx)) is read straight from
// X[i][c][y' * stride - pad + ky][x' * stride - pad + kx], zero outside the map, so the kh * kw-fold copy of
// the input never exists), and optionally by dL/dZ in its native [B][c_out][T] layout.
template <typename T, bool GRAD, bool CONV = false>
__global__ void __launch_bounds__(SIMT_THREADS)
zta_simt_kernel(SimtParams p) {
    __shared__ __align__(16) float Zs[2][SIMT_BK][SIMT_BM];
    __shared__ __align__(16) float As[2][SIMT_BK][SIMT_BN];
    __shared__ float red[32];

    const T* __restrict__ A = static_cast<const T*>(p.A);
    const T* __restrict__ Z = static_cast<const T*>(p.Z);
    const int tid = threadIdx.x;
    const int ty = tid >> 4, tx = tid & 15;          // compute mapping: rows 4*ty.., cols 4*tx..
    const int lk = tid >> 4, lc = (tid & 15) << 2;   // load mapping: slab row lk, columns lc..lc+3

    long row_begin, row_end;
    int tile_first, tile_step;
    if (GRAD) {
        row_begin = (long)blockIdx.y * p.rows_per_split;
        row_end = min(row_begin + p.rows_per_split, p.rows_total);
        tile_first = blockIdx.x; tile_step = gridDim.x;      // gridDim.x == number of tiles
    } else {
        row_begin = (long)blockIdx.y * p.T;
        row_end = row_begin + p.T;
        tile_first = blockIdx.x; tile_step = gridDim.x;      // tiles strided over the split
    }
    const int n_tiles = p.tiles_m * p.tiles_n;
    const int n_slabs = (int)((row_end - row_begin + SIMT_BK - 1) / SIMT_BK);
    float fro = 0.f;

    for (int tile = tile_first; tile < n_tiles; tile += tile_step) {
        const int m0 = (tile / p.tiles_n) * SIMT_BM;
        const int n0 = (tile % p.tiles_n) * SIMT_BN;
        float acc[4][4];
#pragma unroll
        for (int i = 0; i < 4; ++i)
#pragma unroll
            for (int j = 0; j < 4; ++j) acc[i][j] = 0.f;

        float cf = 1.f;
        // CONV: this thread's four patch columns, fixed for the tile: offset inside an example's map and tap
        int coff[4], cky[4], ckx[4];
        if (CONV) {
#pragma unroll
            for (int j = 0; j < 4; ++j) {
                const int n = n0 + lc + j, kk = p.kh * p.kw;
                const int c = n / kk, rem = n - c * kk;
                cky[j] = rem / p.kw; ckx[j] = rem - cky[j] * p.kw;
                coff[j] = (c * p.cH + cky[j]) * p.cW + ckx[j];
            }
        }
        auto fetch = [&](int slab, float4& zr, float4& ar) {
            const long r = row_begin + (long)slab * SIMT_BK + lk;
            const bool ok = r < row_end;
            if (CONV) {
                const int ri = (int)r;                                // B * T < 2^31 (checked by the launcher)
                const int i = ri / p.T, t = ri - i * p.T;
                const int yo = t / p.Wo, xo = t - yo * p.Wo;
                const int y0 = yo * p.stride - p.pad, x0 = xo * p.stride - p.pad;
                const T* xi = A + (size_t)i * p.cC * p.cH * p.cW + (y0 * p.cW + x0);
                float e[4];
#pragma unroll
                for (int j = 0; j < 4; ++j) {
                    const int n = n0 + lc + j;
                    const int y = y0 + cky[j], x = x0 + ckx[j];
                    float v = 0.f;
                    if (ok) {
                        if (n < p.d_in) { if (y >= 0 && y < p.cH && x >= 0 && x < p.cW) v = to_f32(xi[coff[j]]); }
                        else if (n == p.d_in && p.has_bias) v = 1.f;
                    }
                    e[j] = v;
                }
                ar = make_float4(e[0], e[1], e[2], e[3]);
                if (p.z_cm) {
#pragma unroll
                    for (int j = 0; j < 4; ++j) {
                        const int m = m0 + lc + j;
                        e[j] = (ok && m < p.d_out) ? to_f32(Z[((size_t)i * p.d_out + m) * p.T + t]) : 0.f;
                    }
                    zr = make_float4(e[0], e[1], e[2], e[3]);
                } else {
                    zr = simt_load_row4(Z, p.ldz, r, m0 + lc, p.d_out, ok, p.vec_z != 0, false);
                }
            } else {
            zr = simt_load_row4(Z, p.ldz, r, m0 + lc, p.d_out, ok, p.vec_z != 0, false);
            ar = simt_load_row4(A, p.lda, r, n0 + lc, p.d_in, ok, p.vec_a != 0, p.has_bias != 0);
            }
            cf = 1.f;
            if (GRAD) {
                if (ok && p.clip) cf = __ldg(p.clip + r / p.T);
            }
        };
        // the loaded values are first touched here, after the FMAs of the current slab
        auto stash = [&](int buf, const float4& zr, const float4& ar) {
            *reinterpret_cast<float4*>(&Zs[buf][lk][lc]) = make_float4(zr.x * cf, zr.y * cf, zr.z * cf, zr.w * cf);
            *reinterpret_cast<float4*>(&As[buf][lk][lc]) = ar;
        };

        float4 zr, ar;
        if (n_slabs > 0) {
            fetch(0, zr, ar);
            stash(0, zr, ar);
        }
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
            if (more) stash(buf ^ 1, zr, ar);
            __syncthreads();
        }

        if (GRAD) {
#pragma unroll
            for (int i = 0; i < 4; ++i) {
                const int m = m0 + (ty << 2) + i;
                if (m >= p.d_out) continue;
#pragma unroll
                for (int j = 0; j < 4; ++j) {
                    const int n = n0 + (tx << 2) + j;
                    float* dst = nullptr;
                    if (n < p.d_in) dst = p.gW + (size_t)m * p.ldg + n;
                    else if (n == p.d_in && p.has_bias && p.gb) dst = p.gb + m;
                    if (dst) {
                        if (p.use_atomic) atomicAdd(dst, acc[i][j]);
                        else *dst = acc[i][j];
                    }
                }
            }
        } else {
            // out-of-range rows/columns were loaded as zeros, so they add nothing
#pragma unroll
            for (int i = 0; i < 4; ++i)
#pragma unroll
                for (int j = 0; j < 4; ++j) fro = fmaf(acc[i][j], acc[i][j], fro);
        }
    }

    if (!GRAD) {
        fro = block_sum(fro, red);
        if (tid == 0) {
            if (p.use_atomic) atomicAdd(p.sq + blockIdx.y, fro);
            else p.sq[blockIdx.y] = fro;
        }
    }
}

}  // namespace dpclip
