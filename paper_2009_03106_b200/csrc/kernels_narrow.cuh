// Streaming kernel for narrow layers: d_in (+1 with a bias) <= 32 and d_out <= 64,
// e.g. the first 3x3 convolution of an RGB network (d_in = 27, T = H*W large).
//
// Such a layer is pure streaming (a few hundred flops per row, rows of odd
// length that neither TMA nor per-row 128-bit loads can fetch), and a 64 x 64
// tile kernel wastes most of its lanes on it.  Here a lane owns one column n of
// the product Zb^T [A | 1] (d_out accumulators in registers) and a warp walks
// the rows in chunks of 32 (16 when d_out > 32).  With dense rows a chunk of A
// and of Zb is one contiguous run of memory whatever the row length, so the
// warp fetches it with 128-bit loads (all issued before the previous chunk is
// computed, i.e. a whole chunk per warp in flight), parks it in shared memory,
// and then every lane reads its own a[row][n] and the zb row as broadcast
// 128-bit loads.  The sixteen warps of a CTA take interleaved chunks; their
// partial tiles are combined in shared memory at the end.
//
//   NORM: one CTA per example; the tile is squared and summed -> sq[i].
//   GRAD: one CTA per row slice, each row weighted by its example's clip factor
//         (applied to a[row][n] as it is read); the CTA's tile goes to a partial
//         buffer and narrow_reduce_kernel sums the partials in a fixed order and
//         adds the noise (148 CTAs adding onto the same thousand addresses with
//         atomics serialise; without a workspace the atomics remain the fallback).
#pragma once
#include "common.cuh"
#include "kernels_stream.cuh"

namespace dpclip {

constexpr int NARROW_THREADS = 512, NARROW_WARPS = NARROW_THREADS / 32;   // 16 warps: one CTA per SM, latency hidden by warps

struct NarrowParams {
    const void* A; long lda;
    const void* Z; long ldz;
    int T, d_in, d_out, has_bias;
    long rows_total, rows_per_cta;      // GRAD
    const float* clip; float* gW; long ldg; float* gb;
    float* sq;                          // NORM
    float* part;                        // GRAD: per-CTA partial tiles [grid][MAXM][32] instead of atomics (or NULL)
};

template <int MAXM> struct NarrowCfg {
    static constexpr int CH = MAXM == 32 ? 32 : 16;                 // rows per warp chunk
    static constexpr int A_FLOATS = CH * 32, Z_FLOATS = CH * MAXM + 64;   // + slack for reads past short rows
    static constexpr int SMEM_BYTES = NARROW_WARPS * (A_FLOATS + Z_FLOATS) * 4 + MAXM * 33 * 4 + 128;
};

// n consecutive elements starting at src -> fp32 in shared memory, by the whole warp.  128-bit loads
// when src is 16-byte aligned; the loads are issued in `issue`, the values stored in `park`.
template <typename T, int NV> struct ChunkRegs { uint4 v[NV]; };

template <typename T, int NV>
__device__ __forceinline__ void chunk_issue(const T* __restrict__ src, int n, int lane, ChunkRegs<T, NV>& r, bool& vec) {
    constexpr int EPV = 16 / (int)sizeof(T);                        // elements per 128-bit load
    vec = (reinterpret_cast<uintptr_t>(src) & 15) == 0;
    if (vec) {
#pragma unroll
        for (int u = 0; u < NV; ++u) {
            const int e = (u * 32 + lane) * EPV;
            r.v[u] = e + EPV <= n ? __ldg(reinterpret_cast<const uint4*>(src + e)) : make_uint4(0, 0, 0, 0);
        }
    }
}

template <typename T, int NV>
__device__ __forceinline__ void chunk_park(const T* __restrict__ src, int n, int lane, const ChunkRegs<T, NV>& r,
                                           bool vec, float* dst) {
    constexpr int EPV = 16 / (int)sizeof(T);
    int done = 0;
    if (vec) {
#pragma unroll
        for (int u = 0; u < NV; ++u) {
            const int e = (u * 32 + lane) * EPV;
            if (e + EPV <= n) {
                if (sizeof(T) == 4) {
                    *reinterpret_cast<uint4*>(dst + e) = r.v[u];
                } else {
                    const uint32_t w[4] = {r.v[u].x, r.v[u].y, r.v[u].z, r.v[u].w};
                    *reinterpret_cast<float4*>(dst + e) =
                        make_float4(__uint_as_float(w[0] << 16), __uint_as_float(w[0] & 0xFFFF0000u),
                                    __uint_as_float(w[1] << 16), __uint_as_float(w[1] & 0xFFFF0000u));
                    *reinterpret_cast<float4*>(dst + e + 4) =
                        make_float4(__uint_as_float(w[2] << 16), __uint_as_float(w[2] & 0xFFFF0000u),
                                    __uint_as_float(w[3] << 16), __uint_as_float(w[3] & 0xFFFF0000u));
                }
            }
        }
        done = (n / EPV) * EPV;
    }
    for (int e = done + lane; e < n; e += 32) dst[e] = to_f32(src[e]);      // unaligned chunk, or the tail
}

template <typename T, int MAXM, bool GRAD>
__global__ void __launch_bounds__(NARROW_THREADS)
narrow_kernel(NarrowParams p) {
    using Cfg = NarrowCfg<MAXM>;
    constexpr int CH = Cfg::CH;
    constexpr int EPV = 16 / (int)sizeof(T);
    constexpr int NVA = (CH * 32 + 32 * EPV - 1) / (32 * EPV), NVZ = (CH * MAXM + 32 * EPV - 1) / (32 * EPV);
    extern __shared__ __align__(16) float narrow_smem[];
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    float* As = narrow_smem + warp * (Cfg::A_FLOATS + Cfg::Z_FLOATS);
    float* Zs = As + Cfg::A_FLOATS;
    float (*Gs)[33] = reinterpret_cast<float (*)[33]>(narrow_smem + NARROW_WARPS * (Cfg::A_FLOATS + Cfg::Z_FLOATS));
    __shared__ float red[32];

    const T* __restrict__ A = static_cast<const T*>(p.A);
    const T* __restrict__ Z = static_cast<const T*>(p.Z);
    long r0, r1;
    if (GRAD) { r0 = (long)blockIdx.x * p.rows_per_cta; r1 = min(r0 + p.rows_per_cta, p.rows_total); }
    else { r0 = (long)blockIdx.x * p.T; r1 = r0 + p.T; }

    for (int i = threadIdx.x; i < MAXM * 33; i += NARROW_THREADS) (&Gs[0][0])[i] = 0.f;

    float G[MAXM];
#pragma unroll
    for (int m = 0; m < MAXM; ++m) G[m] = 0.f;

    const bool a_lane = lane < p.d_in, one_lane = p.has_bias && lane == p.d_in;
    const bool zvec = (p.d_out & 3) == 0;                          // zb rows start on 16-byte boundaries in smem
    ChunkRegs<T, NVA> ra;
    ChunkRegs<T, NVZ> rz;
    bool va = false, vz = false;
    const long stride = (long)NARROW_WARPS * CH;
    long base = r0 + (long)warp * CH;
    auto rows_of = [&](long b) { return (int)min((long)CH, r1 - b); };
    if (base < r1) {
        const int nr = rows_of(base);
        chunk_issue<T, NVA>(A + (size_t)base * p.lda, nr * p.d_in, lane, ra, va);
        chunk_issue<T, NVZ>(Z + (size_t)base * p.ldz, nr * p.d_out, lane, rz, vz);
    }
    for (; base < r1; base += stride) {
        const int nr = rows_of(base);
        chunk_park<T, NVA>(A + (size_t)base * p.lda, nr * p.d_in, lane, ra, va, As);
        chunk_park<T, NVZ>(Z + (size_t)base * p.ldz, nr * p.d_out, lane, rz, vz, Zs);
        __syncwarp();
        if (base + stride < r1) {                                  // next chunk's loads fly during this chunk's FMAs
            const int nn = rows_of(base + stride);
            chunk_issue<T, NVA>(A + (size_t)(base + stride) * p.lda, nn * p.d_in, lane, ra, va);
            chunk_issue<T, NVZ>(Z + (size_t)(base + stride) * p.ldz, nn * p.d_out, lane, rz, vz);
        }
        int e = GRAD ? (int)(base / p.T) : 0, rem = GRAD ? (int)(base - (long)e * p.T) : 0;
        float c = 1.f;
        if (GRAD) { if (p.clip) c = __ldg(p.clip + e); }
#pragma unroll 4
        for (int r = 0; r < nr; ++r) {
            float ar = a_lane ? As[r * p.d_in + lane] : (one_lane ? 1.f : 0.f);
            if (GRAD) {
                ar *= c;
                if (++rem == p.T) { rem = 0; ++e; if (p.clip && base + r + 1 < r1) c = __ldg(p.clip + e); }
            }
            const float* zr = Zs + r * p.d_out;
            if (zvec) {
#pragma unroll
                for (int m4 = 0; m4 < MAXM / 4; ++m4) {
                    const float4 z4 = *reinterpret_cast<const float4*>(zr + 4 * m4);          // broadcast
                    G[4 * m4 + 0] = fmaf(z4.x, ar, G[4 * m4 + 0]);
                    G[4 * m4 + 1] = fmaf(z4.y, ar, G[4 * m4 + 1]);
                    G[4 * m4 + 2] = fmaf(z4.z, ar, G[4 * m4 + 2]);
                    G[4 * m4 + 3] = fmaf(z4.w, ar, G[4 * m4 + 3]);
                }
            } else {
#pragma unroll
                for (int m = 0; m < MAXM; ++m) G[m] = fmaf(zr[m], ar, G[m]);
            }
        }
        __syncwarp();
    }

    __syncthreads();                                               // Gs zeroed by everyone
#pragma unroll
    for (int m = 0; m < MAXM; ++m)
        if (m < p.d_out) atomicAdd(&Gs[m][lane], G[m]);            // entries m >= d_out hold garbage: never used
    __syncthreads();

    if (GRAD && p.part) {
        float* mine = p.part + (size_t)blockIdx.x * MAXM * 32;
        for (int i = threadIdx.x; i < MAXM * 32; i += NARROW_THREADS) mine[i] = Gs[i >> 5][i & 31];
    } else if (GRAD) {
        for (int i = threadIdx.x; i < p.d_out * 32; i += NARROW_THREADS) {
            const int m = i >> 5, n = i & 31;
            if (n < p.d_in) atomicAdd(p.gW + (size_t)m * p.ldg + n, Gs[m][n]);
            else if (n == p.d_in && p.has_bias && p.gb) atomicAdd(p.gb + m, Gs[m][n]);
        }
    } else {
        float s = 0.f;
        for (int i = threadIdx.x; i < p.d_out * 32; i += NARROW_THREADS) {
            const float v = Gs[i >> 5][i & 31];                    // unused columns hold zeros
            s = fmaf(v, v, s);
        }
        s = block_sum(s, red);
        if (threadIdx.x == 0) p.sq[blockIdx.x] = s;
    }
}

// ---------------------------------------------------------------------------
// fp32 inputs whose chunks start on 16-byte boundaries: the same computation with the chunks copied
// by cp.async straight into a per-warp ring of shared-memory slots (16 rows per chunk, three slots;
// two when d_out > 32).  No staging registers, so several chunks per warp are in flight from the
// first instruction on and the inner loop has registers to keep two rows' operands outstanding (the
// register-staged kernel above stalls on its shared-memory loads for lack of them).
// ---------------------------------------------------------------------------
template <int MAXM, int WARPS_> struct NarrowRingCfg {
    static constexpr int CH = 16;
    // 8 warps: half an SM's shared memory, two CTAs per SM (one computes while the other starts up or winds
    // down); 16 warps: one CTA per SM, for launches with fewer CTAs than SMs (one example per CTA, small B)
    static constexpr int WARPS = WARPS_, THREADS = 32 * WARPS;
    static constexpr int SLOTS = MAXM == 32 ? 3 : 2;
    static constexpr int A_FLOATS = CH * 32, Z_FLOATS = CH * MAXM + 64;      // + slack for reads past short rows
    static constexpr int SLOT_FLOATS = A_FLOATS + Z_FLOATS;
    static constexpr int SMEM_BYTES = WARPS * SLOTS * SLOT_FLOATS * 4 + MAXM * 33 * 4 + 128;
};

__device__ __forceinline__ void cp_async_16(float* smem_dst, const float* gmem_src) {
    asm volatile("cp.async.cg.shared.global [%0], [%1], 16;" ::"r"((uint32_t)__cvta_generic_to_shared(smem_dst)),
                 "l"(gmem_src) : "memory");
}
__device__ __forceinline__ void cp_async_commit() { asm volatile("cp.async.commit_group;" ::: "memory"); }
template <int N> __device__ __forceinline__ void cp_async_wait() { asm volatile("cp.async.wait_group %0;" ::"n"(N) : "memory"); }

// n floats (n % 4 == 0 is copied by cp.async; a remainder of up to 3 floats by plain loads)
__device__ __forceinline__ void ring_issue(float* dst, const float* __restrict__ src, int n, int lane) {
    const int nv = n >> 2;
    for (int v = lane; v < nv; v += 32) cp_async_16(dst + 4 * v, src + 4 * v);
    if (lane < (n & 3)) dst[(nv << 2) + lane] = src[(nv << 2) + lane];
}

template <int MAXM, int WARPS, bool GRAD>
__global__ void __launch_bounds__(32 * WARPS, 16 / WARPS)
narrow_ring_kernel(NarrowParams p) {
    using Cfg = NarrowRingCfg<MAXM, WARPS>;
    constexpr int CH = Cfg::CH, SLOTS = Cfg::SLOTS;
    extern __shared__ __align__(16) float narrow_smem[];
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    float* ring = narrow_smem + warp * SLOTS * Cfg::SLOT_FLOATS;
    float (*Gs)[33] = reinterpret_cast<float (*)[33]>(narrow_smem + Cfg::WARPS * SLOTS * Cfg::SLOT_FLOATS);
    __shared__ float red[32];

    const float* __restrict__ A = static_cast<const float*>(p.A);
    const float* __restrict__ Z = static_cast<const float*>(p.Z);
    long r0, r1;
    if (GRAD) { r0 = (long)blockIdx.x * p.rows_per_cta; r1 = min(r0 + p.rows_per_cta, p.rows_total); }
    else { r0 = (long)blockIdx.x * p.T; r1 = r0 + p.T; }

    const long stride = (long)Cfg::WARPS * CH;
    const long first = r0 + (long)warp * CH;
    auto rows_of = [&](long b) { return b < r1 ? (int)min((long)CH, r1 - b) : 0; };
    auto issue = [&](long b, int slot) {
        const int nr = rows_of(b);
        if (nr > 0) {
            float* dst = ring + slot * Cfg::SLOT_FLOATS;
            ring_issue(dst, A + (size_t)b * p.lda, nr * p.d_in, lane);
            ring_issue(dst + Cfg::A_FLOATS, Z + (size_t)b * p.ldz, nr * p.d_out, lane);
        }
        cp_async_commit();                                        // one group per chunk, empty or not
    };
#pragma unroll
    for (int s = 0; s < SLOTS; ++s) issue(first + s * stride, s);

    for (int i = threadIdx.x; i < MAXM * 33; i += Cfg::THREADS) (&Gs[0][0])[i] = 0.f;

    // Lane (mi, ni) = (lane / 4, lane % 4) owns the MR x 8 block of the tile at rows MR * mi, columns 8 * ni,
    // and the bias sums of its rows.  Per input row: its zb values with one or two 128-bit loads, its eight
    // a values with scalar loads (four distinct addresses per instruction): about 12 cycles of the shared-
    // memory pipe, where one column per lane with the zb row broadcast to all lanes costs 33 (a 128-bit
    // load takes four cycles even when every lane reads the same address) and bound the kernel.  Blocks that
    // hang over the tile (columns >= d_in, rows >= d_out) accumulate whatever lies behind the row and are
    // dropped at the end.
    constexpr int MR = MAXM / 8;
    const int mi = lane >> 2, ni = lane & 3;
    float G[MR][8], gs[MR];
#pragma unroll
    for (int i = 0; i < MR; ++i) {
        gs[i] = 0.f;
#pragma unroll
        for (int j = 0; j < 8; ++j) G[i][j] = 0.f;
    }
    const bool zvec = (p.d_out & 3) == 0;

    int slot = 0;
    for (long base = first; base < r1; base += stride) {
        cp_async_wait<SLOTS - 1>();                                // this chunk has landed (later ones may be in flight)
        __syncwarp();
        const int nr = rows_of(base);
        const float* As = ring + slot * Cfg::SLOT_FLOATS;
        const float* Zs = As + Cfg::A_FLOATS;
        int e = GRAD ? (int)(base / p.T) : 0, rem = GRAD ? (int)(base - (long)e * p.T) : 0;
        float c = 1.f;
        if (GRAD) { if (p.clip) c = __ldg(p.clip + e); }
        // two rows' operands are kept outstanding: while row r is multiplied, row r + 1 is already loaded
        // into the other register set (ping-pong), so the FMAs never wait for shared memory
        auto load_row = [&](int r, float (&z)[MR], float (&a)[8]) {
            const float* zr = Zs + r * p.d_out + MR * mi;
            if (zvec) {
#pragma unroll
                for (int i = 0; i < MR; i += 4) {
                    const float4 z4 = *reinterpret_cast<const float4*>(zr + i);
                    z[i] = z4.x; z[i + 1] = z4.y; z[i + 2] = z4.z; z[i + 3] = z4.w;
                }
            } else {
#pragma unroll
                for (int i = 0; i < MR; ++i) z[i] = zr[i];
            }
            const float* ar = As + r * p.d_in + 8 * ni;
#pragma unroll
            for (int j = 0; j < 8; ++j) a[j] = ar[j];
        };
        auto fma_row = [&](int r, float (&z)[MR], const float (&a)[8]) {
            if (GRAD) {
#pragma unroll
                for (int i = 0; i < MR; ++i) z[i] *= c;
                if (++rem == p.T) { rem = 0; ++e; if (p.clip && base + r + 1 < r1) c = __ldg(p.clip + e); }
            }
#pragma unroll
            for (int i = 0; i < MR; ++i) {
                gs[i] += z[i];
#pragma unroll
                for (int j = 0; j < 8; ++j) G[i][j] = fmaf(z[i], a[j], G[i][j]);
            }
        };
        float z0[MR], z1[MR], a0[8], a1[8];
        if (nr > 0) load_row(0, z0, a0);
#pragma unroll 1
        for (int r = 0; r < nr; r += 2) {
            if (r + 1 < nr) load_row(r + 1, z1, a1);
            fma_row(r, z0, a0);
            if (r + 2 < nr) load_row(r + 2, z0, a0);
            if (r + 1 < nr) fma_row(r + 1, z1, a1);
        }
        __syncwarp();                                              // everyone is done with the slot
        issue(base + SLOTS * stride, slot);
        if (++slot == SLOTS) slot = 0;
    }
    cp_async_wait<0>();

    __syncthreads();                                               // Gs zeroed by everyone
#pragma unroll
    for (int i = 0; i < MR; ++i) {
        const int m = MR * mi + i;
        if (m >= p.d_out) continue;
#pragma unroll
        for (int j = 0; j < 8; ++j)
            if (8 * ni + j < p.d_in) atomicAdd(&Gs[m][8 * ni + j], G[i][j]);
        if (ni == 0 && p.has_bias) atomicAdd(&Gs[m][p.d_in], gs[i]);          // the all-ones column of [A | 1]
    }
    __syncthreads();

    if (GRAD && p.part) {
        float* mine = p.part + (size_t)blockIdx.x * MAXM * 32;
        for (int i = threadIdx.x; i < MAXM * 32; i += Cfg::THREADS) mine[i] = Gs[i >> 5][i & 31];
    } else if (GRAD) {
        for (int i = threadIdx.x; i < p.d_out * 32; i += Cfg::THREADS) {
            const int m = i >> 5, n = i & 31;
            if (n < p.d_in) atomicAdd(p.gW + (size_t)m * p.ldg + n, Gs[m][n]);
            else if (n == p.d_in && p.has_bias && p.gb) atomicAdd(p.gb + m, Gs[m][n]);
        }
    } else {
        float s = 0.f;
        for (int i = threadIdx.x; i < p.d_out * 32; i += Cfg::THREADS) {
            const float v = Gs[i >> 5][i & 31];                    // unused columns hold zeros
            s = fmaf(v, v, s);
        }
        s = block_sum(s, red);
        if (threadIdx.x == 0) p.sq[blockIdx.x] = s;
    }
}

// Second stage of the narrow clipped sum: out[m][n] = sum over the CTAs' partial tiles, + noise.
// One CTA per output row m: 32 columns x 8 groups of partials, combined through shared memory.
struct NarrowReduceParams {
    const float* part; int n_parts, maxm;
    int d_out, d_in, has_bias;
    float* gW; long ldg; float* gb;
    float noise_scale; uint32_t k0, k1; unsigned long long sid_w, sid_b;
};

__global__ void __launch_bounds__(256)
narrow_reduce_kernel(const NarrowReduceParams p) {
    __shared__ float comb[8][32];
    const int m = blockIdx.x, n = threadIdx.x & 31, g = threadIdx.x >> 5;
    const size_t stride = (size_t)p.maxm * 32;
    const float* src = p.part + (size_t)m * 32 + n;
    float acc = 0.f;
    int ks = g;
    for (; ks + 24 < p.n_parts; ks += 32) {                          // four independent loads in flight
        float v[4];
#pragma unroll
        for (int u = 0; u < 4; ++u) v[u] = __ldcs(src + (size_t)(ks + 8 * u) * stride);
        acc += (v[0] + v[1]) + (v[2] + v[3]);
    }
    for (; ks < p.n_parts; ks += 8) acc += __ldcs(src + (size_t)ks * stride);
    comb[g][n] = acc;
    __syncthreads();
    if (g != 0) return;
#pragma unroll
    for (int j = 1; j < 8; ++j) acc += comb[j][n];
    const bool is_bias = n == p.d_in && p.has_bias;
    if (n >= p.d_in && !is_bias) return;
    if (p.noise_scale > 0.f) {
        const size_t e = is_bias ? (size_t)m : (size_t)m * p.d_in + n;
        const unsigned long long sid = is_bias ? p.sid_b : p.sid_w;
        const size_t q = e >> 2;
        PhiloxBlock b = philox_block((uint32_t)q, (uint32_t)(q >> 32), (uint32_t)sid, (uint32_t)(sid >> 32), p.k0, p.k1);
        float za, zb;
        box_muller(b.v[e & 2], b.v[(e & 2) + 1], za, zb);
        acc = fmaf(p.noise_scale, (e & 1) ? zb : za, acc);
    }
    if (is_bias) p.gb[m] = acc; else p.gW[(size_t)m * p.ldg + n] = acc;
}

}  // namespace dpclip
