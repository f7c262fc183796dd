// Narrow layers on the tensor cores, four row groups packed into one instruction (bf16 and fp32):
// d_in (+1 with a bias) <= 32 and d_out <= 32, dense rows, e.g. the first 3x3 convolution of an RGB network.
//
// A 128 x N x 16 MMA costs about 100 clk whatever N is, and a 32 x 28 product fills a sixteenth of it: with one
// such instruction per 16 input rows the instruction count bounds the kernel.  Here a stage of 64 rows is
// split into four groups of 16 rows, and group g goes to the operand COLUMNS 32 g .. 32 g + 31 of both tiles:
//     Zb tile   [16 K-rows][128 M-columns]:  column 32 g + m, K-row k  =  zb[row 16 g + k][m]
//     [A|1] tile [16 K-rows][128 N-columns]: column 32 g + n, K-row k  =  a [row 16 g + k][n]  (n = d_in: ones)
// One 128 x 128 x 16 instruction then computes sixteen 32 x 32 blocks of which the four DIAGONAL ones are
// the products of the four groups (the others pair rows of different groups and are never read): 64 rows per
// instruction instead of 16.  The epilogue adds the four diagonal blocks.
//   bf16: one kind::f16 instruction per stage.  fp32: error-compensated tf32 (x = hi + lo, three products),
//   K = 8 per instruction: six instructions per stage, against 24 without the packing -- which is what makes the
//   tensor cores worth it for fp32 narrow layers at all.  Each diagonal block accumulates a quarter of the rows,
//   and the four are added in fp32, so the accumulator's truncation bias stays below that of a 256-row sum.
// Data path as in kernels_narrow_tc.cuh: one thread bulk-copies 64-row chunks of A and Zb into a ring of raw
// chunks, teams of converter warps re-arrange them into the operand tiles of their own stage slot (fp32: raw
// value = high part, since the tensor core ignores the low 13 mantissa bits; low part into its own plane),
// one thread issues the MMAs, four epilogue warps.
//   The four blocks are added through shared memory.  NORM: item = example; the sum is squared and summed -> sq[i]
//   (atomics).  GRAD: one row slice per CTA, zb scaled by the clip factor during the conversion (bf16: one rounding;
//   fp32: exact to fp32); the sum is the CTA's partial tile for narrow_reduce_kernel.
// Needs 16-byte aligned inputs and T * d_in, T * d_out multiples of 16 bytes' worth of elements.  Every wait is
// bounded; on a timeout the CTA sets the status word and unwinds.
#pragma once
#include "tc_common.cuh"
#include "kernels_tf32.cuh"      // TF32_MASK, mma_tf32_ss helpers

namespace dpclip {
namespace tc {
namespace npk {
constexpr int BK = 64;                           // rows per chunk and per stage (four groups of 16)
constexpr int EPI_WARPS = 4, CONV_WARPS = 12;
constexpr int THREADS = 32 * (2 + EPI_WARPS + CONV_WARPS);     // warp 0 copies, warp 1 MMA, 2..5 epilogue, 6..17 convert
constexpr int RAW_BYTES = 96 * 1024;             // ring of raw chunks
constexpr int MAX_RAW = 24;
constexpr int RED_BYTES = 4 * 32 * 33 * 4;       // NORM: the four diagonal blocks meet here

template <typename T> struct Cfg {
    static constexpr bool F32 = sizeof(T) == 4;
    static constexpr int PLANE_BYTES = 16 * 128 * (int)sizeof(T);          // one operand tile: 16 K-rows x 128 columns
    static constexpr int STAGE_BYTES = (F32 ? 4 : 2) * PLANE_BYTES;         // bf16: Z, A; fp32: Z hi, Z lo, A hi, A lo
    static constexpr int STAGES = F32 ? 3 : 6;                              // = converter teams
    static constexpr int TEAM = CONV_WARPS / STAGES;                        // warps per team (each takes BK / TEAM rows)
    static constexpr int SMEM_BYTES = STAGES * STAGE_BYTES + RAW_BYTES + RED_BYTES + 1024 /*barriers*/ + 1024 /*alignment*/;
};

struct Params {
    const void* A; const void* Z;      // dense rows: row r at A + r * d_in, Z + r * d_out elements
    int T, d_in, d_out, has_bias;
    int n_items;                       // NORM: examples
    long rows_total, rows_per_cta;     // GRAD: one slice per CTA (rows_per_cta a multiple of 32)
    const float* clip;                 // GRAD: [B] or NULL
    float* sq;                         // NORM: [B], pre-zeroed
    float* part;                       // GRAD: [grid][32][32] partial tiles
    int* status;
};

// byte offset of (K-row k, column c) in a [16][128] operand tile
__device__ __forceinline__ uint32_t off_bf16(int k, int c) {     // MN-major, 128-byte swizzle, 64-column chunks of 2048 bytes
    return (uint32_t)((c >> 6) * 2048 + k * 128 + (((((c & 63) >> 3) ^ (k & 7)) << 4) | ((c & 7) << 1)));
}
__device__ __forceinline__ uint32_t off_f32(int k, int c) {      // MN-major 32-bit, 128-byte swizzle on 32-byte atoms
    return (uint32_t)((c >> 5) * 2048 + (k >> 2) * 512 + (k & 3) * 128 + (((((c & 31) >> 3) ^ (k & 3)) << 5) | ((c & 7) << 2)));
}
__device__ __forceinline__ void bulk_load(void* smem_dst, const void* gmem_src, uint32_t bytes, uint64_t* bar) {
    asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];"
                 ::"r"(smem_u32(smem_dst)), "l"(gmem_src), "r"(bytes), "r"(smem_u32(bar)) : "memory");
}
}  // namespace npk

template <typename T, bool GRAD>
__global__ void __launch_bounds__(npk::THREADS, 1)
narrow_pack_kernel(const npk::Params p) {
    using namespace npk;
    using C = Cfg<T>;
    constexpr bool F32 = C::F32;
    constexpr int ES = (int)sizeof(T), STAGES = C::STAGES, STAGE_BYTES = C::STAGE_BYTES, PLANE = C::PLANE_BYTES, TEAM = C::TEAM;
    extern __shared__ uint8_t smem_raw[];
    uint8_t* smem = smem_raw + ((1024u - (smem_u32(smem_raw) & 1023u)) & 1023u);
    uint8_t* raw = smem + STAGES * STAGE_BYTES;
    float* red = reinterpret_cast<float*>(raw + RAW_BYTES);
    uint64_t* full = reinterpret_cast<uint64_t*>(raw + RAW_BYTES + RED_BYTES);
    uint64_t* empty = full + STAGES;
    uint64_t* raw_full = empty + STAGES;
    uint64_t* raw_empty = raw_full + MAX_RAW;
    uint64_t* acc_full = raw_empty + MAX_RAW;
    uint64_t* acc_empty = acc_full + 2;
    uint64_t* red_full = acc_empty + 2;          // NORM: the four blocks of an item are in `red`
    uint64_t* red_empty = red_full + 1;          // ... and have been summed
    uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(red_empty + 1);
    volatile int* abort_flag = reinterpret_cast<volatile int*>(tmem_slot + 1);

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int za = p.d_out, aa = p.d_in;
    const int a_chunk = BK * aa * ES, z_chunk = BK * za * ES, chunk_bytes = a_chunk + z_chunk;
    const int n_raw = min(MAX_RAW, RAW_BYTES / chunk_bytes) / STAGES * STAGES;      // a multiple of the teams: see below

    if (threadIdx.x == 0) {
        DPCLIP_TRACE_AT(0, 254);
        for (int s = 0; s < STAGES; ++s) { mbar_init(&full[s], TEAM); mbar_init(&empty[s], 1); }
        for (int s = 0; s < MAX_RAW; ++s) { mbar_init(&raw_full[s], 1); mbar_init(&raw_empty[s], TEAM); }
        for (int b = 0; b < 2; ++b) { mbar_init(&acc_full[b], 1); mbar_init(&acc_empty[b], EPI_WARPS); }
        mbar_init(red_full, EPI_WARPS); mbar_init(red_empty, EPI_WARPS);
        *abort_flag = 0;
        mbar_fence_init();
    }
    __syncthreads();

    const int n_items = GRAD ? 1 : p.n_items;
    const int item0 = GRAD ? 0 : blockIdx.x, item_step = GRAD ? 1 : gridDim.x;
    auto item_rows = [&](int item, long& r0, long& r1) {
        if (GRAD) { r0 = (long)blockIdx.x * p.rows_per_cta; r1 = min(r0 + p.rows_per_cta, p.rows_total); }
        else { r0 = (long)item * p.T; r1 = r0 + p.T; }
    };

    uint32_t tmem_base = 0;
    if (warp == 0) {
        // ------------------------------------------------ copy: raw chunks, as far ahead as the ring allows; takes no
        // part in the set-up of the other warps
        if (lane == 0) {
            int slot = 0; uint32_t phase = 0;
            bool ok = true;
            const uint8_t* Ab = static_cast<const uint8_t*>(p.A);
            const uint8_t* Zb = static_cast<const uint8_t*>(p.Z);
            for (int item = item0; item < n_items && ok; item += item_step) {
                long r0, r1; item_rows(item, r0, r1);
                for (long rb = r0; rb < r1; rb += BK) {
                    const int nr = (int)min((long)BK, r1 - rb);
                    ok = mbar_wait(&raw_empty[slot], phase ^ 1, abort_flag, p.status);
                    if (!ok) break;
                    uint8_t* dst = raw + slot * chunk_bytes;
                    mbar_arrive_expect_tx(&raw_full[slot], (uint32_t)(nr * (aa + za) * ES));
                    bulk_load(dst, Ab + (size_t)rb * aa * ES, (uint32_t)(nr * aa * ES), &raw_full[slot]);
                    bulk_load(dst + a_chunk, Zb + (size_t)rb * za * ES, (uint32_t)(nr * za * ES), &raw_full[slot]);
                    if (++slot == n_raw) { slot = 0; phase ^= 1; }
                }
            }
        }
    } else {
        constexpr int OTHERS = THREADS - 32;
        auto sync_others = [&]() { asm volatile("bar.sync 1, %0;" ::"r"(OTHERS) : "memory"); };
        // operand tiles start all zero; the converters only ever write the real columns of each group, so the
        // padding stays zero.  The bias column (ones) of every group is set once.
        for (int i = threadIdx.x - 32; i < STAGES * STAGE_BYTES / 16; i += OTHERS)
            reinterpret_cast<uint4*>(smem)[i] = make_uint4(0, 0, 0, 0);
        sync_others();
        if (p.has_bias)
            for (int i = threadIdx.x - 32; i < STAGES * 64; i += OTHERS) {
                const int s = i >> 6, g = (i >> 4) & 3, k = i & 15;
                uint8_t* at = smem + s * STAGE_BYTES + (F32 ? 2 : 1) * PLANE;       // A (high) plane
                if (F32) *reinterpret_cast<float*>(at + off_f32(k, 32 * g + aa)) = 1.f;
                else *reinterpret_cast<__nv_bfloat16*>(at + off_bf16(k, 32 * g + aa)) = __float2bfloat16_rn(1.f);
            }
        if (warp == 1) { tmem_alloc(tmem_slot, 256); tmem_relinquish(); }
        fence_proxy_async_smem();
        tc_fence_before_sync();
        sync_others();
        tc_fence_after_sync();
        tmem_base = *tmem_slot;
    }
    if (warp == 1) {
        // ------------------------------------------------ MMA issuer
        if (lane == 0) {
            constexpr uint32_t idesc = F32 ? make_idesc_tf32(128, 128, 1, 1) : make_idesc_bf16(128, 128, 1, 1);
            int stage = 0; uint32_t phase = 0; int it = 0;
            bool ok = true;
            [[maybe_unused]] int tr = 0;
            DPCLIP_TRACE_AT(0, 255);
            for (int item = item0; item < n_items && ok; item += item_step, ++it) {
                long r0, r1; item_rows(item, r0, r1);
                const int nkb = (int)((r1 - r0 + BK - 1) / BK);
                const int buf = it & 1;
                ok = mbar_wait(&acc_empty[buf], ((it >> 1) & 1) ^ 1, abort_flag, p.status);
                if (!ok) break;
                tc_fence_after_sync();
                const uint32_t d_tmem = tmem_base + buf * 128;
                for (int kb = 0; kb < nkb; ++kb) {
                    ok = mbar_wait(&full[stage], phase, abort_flag, p.status);
                    if (!ok) break;
                    DPCLIP_TRACE_AT(2, tr); ++tr;
                    tc_fence_after_sync();
                    const uint32_t base = smem_u32(smem + stage * STAGE_BYTES);
                    if (F32) {
#pragma unroll
                        for (int k8 = 0; k8 < 2; ++k8) {
                            // MN-major fp32 operands, 128-byte swizzle on 32-byte atoms: 32-column chunks 2048 bytes apart,
                            // 4-row groups 512 bytes apart, 8 rows per K = 8 instruction; small terms first
                            const uint64_t zh = make_smem_desc_sw128_atom32(base + k8 * 1024, 2048, 512);
                            const uint64_t zl = make_smem_desc_sw128_atom32(base + PLANE + k8 * 1024, 2048, 512);
                            const uint64_t ah = make_smem_desc_sw128_atom32(base + 2 * PLANE + k8 * 1024, 2048, 512);
                            const uint64_t al = make_smem_desc_sw128_atom32(base + 3 * PLANE + k8 * 1024, 2048, 512);
                            mma_tf32_ss(d_tmem, zl, ah, idesc, (kb == 0 && k8 == 0) ? 0u : 1u);
                            mma_tf32_ss(d_tmem, zh, al, idesc, 1u);
                            mma_tf32_ss(d_tmem, zh, ah, idesc, 1u);
                        }
                    } else {
                        // MN-major bf16, 128-byte swizzle: 64-column chunks 2048 bytes apart, 8-row groups 1024 bytes apart
                        const uint64_t dz = make_smem_desc_sw128(base, 2048, 1024);
                        const uint64_t da = make_smem_desc_sw128(base + PLANE, 2048, 1024);
                        mma_bf16_ss(d_tmem, dz, da, idesc, kb == 0 ? 0u : 1u);
                    }
                    mma_commit(&empty[stage]);
                    if (++stage == STAGES) { stage = 0; phase ^= 1; }
                }
                if (!ok) break;
                mma_commit(&acc_full[buf]);
            }
        }
    } else if (warp >= 2 && warp < 2 + EPI_WARPS) {
        // ------------------------------------------------ epilogue: warp q = w % 4 reads tensor-memory lanes 32 q .. (the
        // output rows of group q) and, of their 128 columns, the 32 of the diagonal block
        const int q = warp & 3;
        int it = 0;
        for (int item = item0; item < n_items; item += item_step, ++it) {
            const int buf = it & 1;
            if (!mbar_wait(&acc_full[buf], (it >> 1) & 1, abort_flag, p.status)) break;
            if (threadIdx.x == 64) DPCLIP_TRACE_AT(3, it);
            tc_fence_after_sync();
            uint32_t v[32];
            tmem_ld_32x32(tmem_base + ((uint32_t)(q * 32) << 16) + buf * 128 + q * 32, v);
            tmem_ld_wait();
            tc_fence_before_sync();
            __syncwarp();
            if (lane == 0) mbar_arrive(&acc_empty[buf]);
            // the four blocks meet in shared memory; warp q then takes rows 8 q .. 8 q + 7 of their sum
            if (!mbar_wait(red_empty, (it & 1) ^ 1, abort_flag, p.status)) break;
            float* mine = red + (q * 32 + lane) * 33;
#pragma unroll
            for (int j = 0; j < 32; ++j) mine[j] = __uint_as_float(v[j]);
            __syncwarp();
            if (lane == 0) mbar_arrive(red_full);
            if (!mbar_wait(red_full, it & 1, abort_flag, p.status)) break;
            float s = 0.f;
#pragma unroll
            for (int m = 8 * q; m < 8 * q + 8; ++m) {
                const float x = (red[(0 * 32 + m) * 33 + lane] + red[(1 * 32 + m) * 33 + lane]) +
                                (red[(2 * 32 + m) * 33 + lane] + red[(3 * 32 + m) * 33 + lane]);
                if (GRAD) p.part[((size_t)blockIdx.x * 32 + m) * 32 + lane] = x;      // the CTA's partial tile
                else s = fmaf(x, x, s);
            }
            __syncwarp();
            if (lane == 0) mbar_arrive(red_empty);
            if (!GRAD) {
                s = warp_sum(s);
                if (lane == 0) atomicAdd(p.sq + item, s);
            }
        }
    } else if (warp >= 2 + EPI_WARPS) {
        // ------------------------------------------------ convert: team f takes the chunks f, f + STAGES, ... of the CTA's
        // chunk sequence into its own stage slot (and owns the raw slots s with s % STAGES == f: the ring is cut into
        // a multiple of STAGES chunks, so a barrier's phases are seen by the same consumers in order); member h of the
        // team converts rows h * RW .. of the chunk: whole 16-row groups
        constexpr int RW = BK / TEAM, EPV = 16 / ES;               // rows per warp; elements per 16-byte vector
        const int cw = warp - (2 + EPI_WARPS), f = cw / TEAM, h = cw - f * TEAM;
        const bool z_vec = (za % EPV) == 0;
        const int vpr = za / EPV;                                  // vectors per zb row (z_vec)
        uint8_t* zt = smem + f * STAGE_BYTES;                      // Z (high) plane; fp32: + PLANE = low plane
        uint8_t* at = zt + (F32 ? 2 : 1) * PLANE;                  // A (high) plane; fp32: + PLANE = low plane
        int seq = 0;
        uint32_t my_phase = 0;
        bool ok = true;
        for (int item = item0; item < n_items && ok; item += item_step) {
            long r0, r1; item_rows(item, r0, r1);
            const int nkb = (int)((r1 - r0 + BK - 1) / BK);
            int kb = (f - seq) % STAGES; if (kb < 0) kb += STAGES;
            for (; kb < nkb; kb += STAGES) {
                const int gs = seq + kb;
                const int rslot = gs % n_raw; const uint32_t rphase = (uint32_t)((gs / n_raw) & 1);
                const long rb = r0 + (long)kb * BK;
                const int nr = (int)min((long)BK, r1 - rb);
                int e0 = 0, rem0 = 0;
                if (GRAD && p.clip) { e0 = (int)(rb / p.T); rem0 = (int)(rb - (long)e0 * p.T); }
                auto factor = [&](int r) {
                    int e = e0, x = rem0 + r;
                    while (x >= p.T) { x -= p.T; ++e; }
                    return __ldg(p.clip + e);
                };
                ok = mbar_wait(&raw_full[rslot], rphase, abort_flag, p.status);
                if (ok) ok = mbar_wait(&empty[f], my_phase ^ 1, abort_flag, p.status);
                if (!ok) break;
                my_phase ^= 1;
                if (cw == 0 && lane == 0) DPCLIP_TRACE_AT(1, 2 * (gs / STAGES));
                const uint8_t* ra = raw + rslot * chunk_bytes;
                const uint8_t* rz = ra + a_chunk;
                // ---- [A|1]: lane = column c; the 16 rows of group grp go to tile column 32 grp + c, K-rows 0 .. 15.
                // Sixteen loads, then sixteen stores (the compiler cannot tell the raw ring from the tile).
                if (lane < aa) {
#pragma unroll
                    for (int b16 = 0; b16 < RW / 16; ++b16) {
                        const int grp = h * (RW / 16) + b16, rbase = grp * 16;
                        if (rbase >= nr) break;
                        const T* src = reinterpret_cast<const T*>(ra) + (size_t)rbase * aa + lane;
                        if (F32) {
                            const uint32_t boff = (uint32_t)(grp * 2048 + ((lane & 7) << 2)), unit = lane >> 3;
                            uint32_t v[16];
#pragma unroll
                            for (int k = 0; k < 16; ++k) v[k] = rbase + k < nr ? reinterpret_cast<const uint32_t*>(src)[k * aa] : 0u;
#pragma unroll
                            for (int k = 0; k < 16; ++k) {
                                const uint32_t o = boff + (k >> 2) * 512 + (k & 3) * 128 + ((unit ^ (k & 3)) << 5);
                                *reinterpret_cast<uint32_t*>(at + o) = v[k];
                                *reinterpret_cast<float*>(at + PLANE + o) = __uint_as_float(v[k]) - __uint_as_float(v[k] & t32::TF32_MASK);
                            }
                        } else {
                            const uint32_t boff = (uint32_t)((grp >> 1) * 2048 + ((lane & 7) << 1)), unit = 4 * (grp & 1) + (lane >> 3);
                            unsigned short v[16];
#pragma unroll
                            for (int k = 0; k < 16; ++k) v[k] = rbase + k < nr ? reinterpret_cast<const unsigned short*>(src)[k * aa] : (unsigned short)0;
#pragma unroll
                            for (int k = 0; k < 16; ++k)
                                *reinterpret_cast<unsigned short*>(at + boff + k * 128 + ((unit ^ (k & 7)) << 4)) = v[k];
                        }
                    }
                }
                // ---- Zb: rows past the end of the item are stored as zeros
                if (z_vec) {
                    const int v_begin = h * RW * vpr, v_end = (h + 1) * RW * vpr, nvalid = nr * vpr;
                    for (int v0 = v_begin + lane; v0 < v_end; v0 += 128) {          // four vectors per lane at a time
                        uint4 w[4];
#pragma unroll
                        for (int u = 0; u < 4; ++u) {
                            const int v = v0 + 32 * u;
                            w[u] = (v < v_end && v < nvalid) ? *reinterpret_cast<const uint4*>(rz + (size_t)v * 16) : make_uint4(0, 0, 0, 0);
                        }
#pragma unroll
                        for (int u = 0; u < 4; ++u) {
                            const int v = v0 + 32 * u;
                            if (v >= v_end) continue;
                            const int r = v / vpr, c = 32 * (r >> 4) + (v - r * vpr) * EPV, k = r & 15;
                            uint32_t* ww = reinterpret_cast<uint32_t*>(&w[u]);
                            if (F32) {
                                float x[4] = {__uint_as_float(ww[0]), __uint_as_float(ww[1]), __uint_as_float(ww[2]), __uint_as_float(ww[3])};
                                if (GRAD && p.clip && v < nvalid) {
                                    const float cf = factor(r);
#pragma unroll
                                    for (int j = 0; j < 4; ++j) x[j] *= cf;
                                }
                                const uint32_t o = off_f32(k, c);
                                *reinterpret_cast<float4*>(zt + o) = make_float4(x[0], x[1], x[2], x[3]);
                                float lo[4];
#pragma unroll
                                for (int j = 0; j < 4; ++j) lo[j] = x[j] - __uint_as_float(__float_as_uint(x[j]) & t32::TF32_MASK);
                                *reinterpret_cast<float4*>(zt + PLANE + o) = make_float4(lo[0], lo[1], lo[2], lo[3]);
                            } else {
                                if (GRAD && p.clip && v < nvalid) {
                                    const float cf = factor(r);
                                    if (cf != 1.0f) {
#pragma unroll
                                        for (int j = 0; j < 4; ++j) {
                                            const __nv_bfloat162 hh = __floats2bfloat162_rn(__uint_as_float(ww[j] << 16) * cf,
                                                                                             __uint_as_float(ww[j] & 0xFFFF0000u) * cf);
                                            ww[j] = *reinterpret_cast<const uint32_t*>(&hh);
                                        }
                                    }
                                }
                                *reinterpret_cast<uint4*>(zt + off_bf16(k, c)) = w[u];
                            }
                        }
                    }
                } else {
                    const T* zsrc = reinterpret_cast<const T*>(rz);
                    for (int idx = h * RW * za + lane; idx < (h + 1) * RW * za; idx += 32) {
                        const int r = idx / za, c = 32 * (r >> 4) + (idx - r * za), k = r & 15;
                        float x = r < nr ? to_f32(zsrc[idx]) : 0.f;
                        if (GRAD && p.clip && r < nr) x *= factor(r);
                        if (F32) {
                            const uint32_t o = off_f32(k, c);
                            *reinterpret_cast<float*>(zt + o) = x;
                            *reinterpret_cast<float*>(zt + PLANE + o) = x - __uint_as_float(__float_as_uint(x) & t32::TF32_MASK);
                        } else {
                            *reinterpret_cast<__nv_bfloat16*>(zt + off_bf16(k, c)) = __float2bfloat16_rn(x);
                        }
                    }
                }
                fence_proxy_async_smem();
                __syncwarp();
                if (lane == 0) { mbar_arrive(&full[f]); mbar_arrive(&raw_empty[rslot]); }
                if (cw == 0 && lane == 0) DPCLIP_TRACE_AT(1, 2 * (gs / STAGES) + 1);
            }
            seq += nkb;
        }
    }

    // ---------------------------------------------------- teardown
    if (*abort_flag) {
        for (int i = 0; i < 64; ++i) __nanosleep(1000);
    }
    tc_fence_before_sync();
    __syncthreads();
    if (warp == 1) { tc_fence_after_sync(); tmem_dealloc(tmem_base, 256); }
}

}  // namespace tc
}  // namespace dpclip
