// Narrow layers on the tensor cores (bf16): d_in (+1 with a bias) <= 32, d_out <= 64, dense rows --
// e.g. the first 3x3 convolution of an RGB network (d_in = 27, T = H*W large).
//
// The fp32-ALU streaming kernels (kernels_narrow.cuh) spend ~40 issue slots and 12-33 cycles of the
// shared-memory pipe per input row and warp; with one example (or row slice) per SM that is 17-20 us for
// the 1024 rows of a 32 x 32 image, whatever the memory system does.  The contraction itself is tiny, so
// here it goes to the tensor cores and the SM's threads only re-arrange data that is already on chip:
//   * rows of 54 bytes cannot be fetched as TMA tiles, but a run of dense rows is one contiguous run of
//     bytes: one thread copies the item's A and Zb bytes, 64 rows at a time, into a ring of raw chunks in
//     shared memory with untiled bulk copies (cp.async.bulk; all chunks of a 1024-row example are
//     requested at once, so the HBM latency is paid once per item, not once per block and warp);
//   * twelve converter warps (six pairs) turn raw chunks into MN-major 128-byte-swizzled operand tiles in their own
//     stage slots (shared memory to shared memory: lane = column for [A|1], 128-bit vectors for Zb):
//         Zb tile    M = 128: d_out real columns in the first 64-column chunk, the rest zero; the
//                    descriptor's chunk stride is 0, so rows 64..127 re-read the chunk and are never used
//         [A|1] tile N = 64: d_in real columns, then the all-ones bias column, the rest zero
//     (the padding is zeroed once and never written);
//   * one thread issues four 128 x 64 x 16 MMAs per 64-row stage into a 64-column accumulator in tensor
//     memory (two buffers); four epilogue warps.
//   NORM: one item per example; the epilogue squares and sums the 64 x 32 block that holds the example's
//         gradient (the padding is exactly zero), so the per-example gradient never leaves the SM.
//   GRAD: one row slice per CTA, Zb scaled by the example's clip factor during the conversion (fp32
//         product, one rounding to bf16); the tile goes to the partial buffer that narrow_reduce_kernel sums.
// Needs 16-byte aligned inputs and T * d_in, T * d_out multiples of 8 (every item and chunk then starts and
// ends on a 16-byte boundary).  Every wait is bounded; on a timeout the CTA sets the status word and unwinds.
#pragma once
#include "tc_common.cuh"

namespace dpclip {
namespace tc {
namespace ntc {
constexpr int BK = 64;                           // rows per chunk and per stage
constexpr int Z_BYTES = BK * 128, A_BYTES = BK * 128;
constexpr int STAGE_BYTES = Z_BYTES + A_BYTES;   // 16 KB
constexpr int CONV_PAIRS = 6, EPI_WARPS = 4;
// Converter pair f (two warps, each takes 32 of a chunk's 64 rows) owns stage slot f and every raw slot s with
// s % 6 == f (the ring is cut into a multiple of 6 chunks; chunk g of the CTA's sequence -> pair g % 6), so the
// phases of a barrier are seen by the same consumers in order: a parity wait cannot tell a barrier that is two
// phases behind from one that is done.
constexpr int STAGES = CONV_PAIRS;
constexpr int THREADS = 32 * (2 + EPI_WARPS + 2 * CONV_PAIRS);     // warp 0 copies, warp 1 MMA, 2..5 epilogue, 6..17 convert
constexpr int RAW_BYTES = 96 * 1024;             // ring of raw chunks
constexpr int MAX_RAW = 24;                      // most raw chunks the ring is cut into
constexpr int SMEM_BYTES = STAGES * STAGE_BYTES + RAW_BYTES + 1024 /*barriers*/ + 1024 /*alignment*/;
constexpr int ACC_COLS = 64;                     // accumulator columns per buffer (N)

struct Params {
    const __nv_bfloat16* A; const __nv_bfloat16* Z;    // dense rows: row r at A + r * d_in, Z + r * d_out
    int T, d_in, d_out, has_bias;
    int n_items;                       // NORM: examples
    long rows_total, rows_per_cta;     // GRAD: one slice per CTA (rows_per_cta a multiple of 32)
    const float* clip;                 // GRAD: [B] or NULL
    float* sq;                         // NORM: [B] (pre-zeroed when d_out > 32)
    float* part;                       // GRAD: [grid][part_m][32] partial tiles
    int part_m;                        // rows of a partial tile (32 or 64)
    int* status;
};

// byte offset of element (row k, column c) inside a 64-column MN-major chunk
__device__ __forceinline__ uint32_t mn_off(int k, int c) {
    return (uint32_t)(k * 128 + ((((c >> 3) ^ (k & 7)) << 4) | ((c & 7) << 1)));
}

// contiguous bytes global -> shared, completion counted on `bar` (addresses and size multiples of 16)
__device__ __forceinline__ void bulk_load(void* smem_dst, const void* gmem_src, uint32_t bytes, uint64_t* bar) {
    asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];"
                 ::"r"(smem_u32(smem_dst)), "l"(gmem_src), "r"(bytes), "r"(smem_u32(bar)) : "memory");
}
}  // namespace ntc

template <bool GRAD>
__global__ void __launch_bounds__(ntc::THREADS, 1)
narrow_tc_kernel(const ntc::Params p) {
    using namespace ntc;
    extern __shared__ uint8_t smem_raw[];
    uint8_t* smem = smem_raw + ((1024u - (smem_u32(smem_raw) & 1023u)) & 1023u);   // 1024-byte aligned; an offset from the array keeps the accesses in the shared state space
    uint8_t* raw = smem + STAGES * STAGE_BYTES;
    uint64_t* full = reinterpret_cast<uint64_t*>(raw + RAW_BYTES);       // operand stage converted
    uint64_t* empty = full + STAGES;                                      // operand stage consumed by the MMAs
    uint64_t* raw_full = empty + STAGES;                                  // raw chunk landed
    uint64_t* raw_empty = raw_full + MAX_RAW;                             // raw chunk converted
    uint64_t* acc_full = raw_empty + MAX_RAW;
    uint64_t* acc_empty = acc_full + 2;
    uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(acc_empty + 2);
    volatile int* abort_flag = reinterpret_cast<volatile int*>(tmem_slot + 1);

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int za = p.d_out, aa = p.d_in;
    // a raw chunk holds BK rows of A, then BK rows of Zb; the ring is cut into as many as fit
    const int a_chunk = BK * aa * 2, z_chunk = BK * za * 2, chunk_bytes = a_chunk + z_chunk;
    const int n_raw = min(MAX_RAW, RAW_BYTES / chunk_bytes) / CONV_PAIRS * CONV_PAIRS;      // >= 6: a chunk is at most 12 KB

    if (threadIdx.x == 0) {
        DPCLIP_TRACE_AT(0, 254);
        for (int s = 0; s < STAGES; ++s) { mbar_init(&full[s], 2); mbar_init(&empty[s], 1); }
        for (int s = 0; s < MAX_RAW; ++s) { mbar_init(&raw_full[s], 1); mbar_init(&raw_empty[s], 2); }
        for (int b = 0; b < 2; ++b) { mbar_init(&acc_full[b], 1); mbar_init(&acc_empty[b], EPI_WARPS); }
        *abort_flag = 0;
        mbar_fence_init();
    }
    __syncthreads();

    // items of this CTA: NORM = examples blockIdx.x, + gridDim.x, ...; GRAD = its one row slice
    const int n_items = GRAD ? 1 : p.n_items;
    const int item0 = GRAD ? 0 : blockIdx.x, item_step = GRAD ? 1 : gridDim.x;
    auto item_rows = [&](int item, long& r0, long& r1) {
        if (GRAD) { r0 = (long)blockIdx.x * p.rows_per_cta; r1 = min(r0 + p.rows_per_cta, p.rows_total); }
        else { r0 = (long)item * p.T; r1 = r0 + p.T; }
    };

    // ------------------------------------------------ copy (warp 0, one thread): raw chunks, as far ahead as the ring
    // allows.  It starts at once (the raw ring needs no preparation) and takes no part in the set-up of the
    // other warps, which meet at a named barrier of their own.
    uint32_t tmem_base = 0;
    if (warp == 0) {
        if (lane == 0) {
            int slot = 0; uint32_t phase = 0;
            bool ok = true;
            for (int item = item0; item < n_items && ok; item += item_step) {
                long r0, r1; item_rows(item, r0, r1);
                for (long rb = r0; rb < r1; rb += BK) {
                    const int nr = (int)min((long)BK, r1 - rb);
                    ok = mbar_wait(&raw_empty[slot], phase ^ 1, abort_flag, p.status);
                    if (!ok) break;
                    uint8_t* dst = raw + slot * chunk_bytes;
                    mbar_arrive_expect_tx(&raw_full[slot], (uint32_t)(nr * (aa + za) * 2));
                    bulk_load(dst, p.A + (size_t)rb * aa, (uint32_t)(nr * aa * 2), &raw_full[slot]);
                    bulk_load(dst + a_chunk, p.Z + (size_t)rb * za, (uint32_t)(nr * za * 2), &raw_full[slot]);
                    if (++slot == n_raw) { slot = 0; phase ^= 1; }
                }
            }
        }
    } else {
        constexpr int OTHERS = THREADS - 32;
        auto sync_others = [&]() { asm volatile("bar.sync 1, %0;" ::"r"(OTHERS) : "memory"); };
        // operand tiles start all zero; the converters only ever write the real columns, so the padding stays
        // zero for the whole kernel.  The bias column of [A|1] is set once.
        for (int i = threadIdx.x - 32; i < STAGES * STAGE_BYTES / 16; i += OTHERS)
            reinterpret_cast<uint4*>(smem)[i] = make_uint4(0, 0, 0, 0);
        sync_others();
        if (p.has_bias)
            for (int i = threadIdx.x - 32; i < STAGES * BK; i += OTHERS) {
                const int s = i / BK, k = i - s * BK;
                *reinterpret_cast<__nv_bfloat16*>(smem + s * STAGE_BYTES + Z_BYTES + mn_off(k, aa)) = __float2bfloat16_rn(1.f);
            }
        if (warp == 1) { tmem_alloc(tmem_slot, 2 * ACC_COLS); tmem_relinquish(); }
        fence_proxy_async_smem();
        tc_fence_before_sync();
        sync_others();
        tc_fence_after_sync();
        tmem_base = *tmem_slot;
    }

    if (warp == 1) {
        // ------------------------------------------------ MMA issuer
        if (lane == 0) {
            constexpr uint32_t idesc = make_idesc_bf16(128, ACC_COLS, 1, 1);
            int stage = 0; uint32_t phase = 0; int it = 0;
            bool ok = true;
            [[maybe_unused]] int tr = 0;
            DPCLIP_TRACE_AT(0, 255);
            for (int item = item0; item < n_items && ok; item += item_step, ++it) {
                long r0, r1; item_rows(item, r0, r1);
                const int nkb = (int)((r1 - r0 + BK - 1) / BK);
                const int buf = it & 1; const uint32_t acc_phase = (it >> 1) & 1;
                ok = mbar_wait(&acc_empty[buf], acc_phase ^ 1, abort_flag, p.status);
                if (!ok) break;
                tc_fence_after_sync();
                for (int kb = 0; kb < nkb; ++kb) {
                    ok = mbar_wait(&full[stage], phase, abort_flag, p.status);
                    if (!ok) break;
                    DPCLIP_TRACE_AT(2, tr); ++tr;
                    tc_fence_after_sync();
                    const uint32_t zb = smem_u32(smem + stage * STAGE_BYTES), ab = zb + Z_BYTES;
#pragma unroll
                    for (int k16 = 0; k16 < BK / 16; ++k16) {
                        // MN-major, 128-byte swizzle: 8-row groups 1024 bytes apart, 16 rows = 2048 bytes; chunk
                        // stride 0 for Zb (see the header), unused for the single chunk of [A|1]
                        const uint64_t dz = make_smem_desc_sw128(zb + k16 * 2048, 0, 1024);
                        const uint64_t da = make_smem_desc_sw128(ab + k16 * 2048, BK * 128, 1024);
                        mma_bf16_ss(tmem_base + buf * ACC_COLS, dz, da, idesc, (kb == 0 && k16 == 0) ? 0u : 1u);
                    }
                    mma_commit(&empty[stage]);
                    if (++stage == STAGES) { stage = 0; phase ^= 1; }
                }
                if (!ok) break;
                mma_commit(&acc_full[buf]);
            }
        }
    } else if (warp >= 2 && warp < 2 + EPI_WARPS) {
        // ------------------------------------------------ epilogue: warp w reads tensor-memory lanes 32 * (w % 4) ..
        const int quarter = warp & 3;
        int it = 0;
        for (int item = item0; item < n_items; item += item_step, ++it) {
            const int buf = it & 1; const uint32_t acc_phase = (it >> 1) & 1;
            if (!mbar_wait(&acc_full[buf], acc_phase, abort_flag, p.status)) break;
            if (threadIdx.x == 64) DPCLIP_TRACE_AT(3, it);
            tc_fence_after_sync();
            if (quarter * 32 < za) {                           // lanes of this quarter hold output rows m = 32 q + lane
                uint32_t v[32];
                tmem_ld_32x32(tmem_base + ((uint32_t)(quarter * 32) << 16) + buf * ACC_COLS, v);
                tmem_ld_wait();
                if (GRAD) {
                    const int m = quarter * 32 + lane;
                    if (m < p.part_m) {
                        float4* dst = reinterpret_cast<float4*>(p.part + ((size_t)blockIdx.x * p.part_m + m) * 32);
#pragma unroll
                        for (int j = 0; j < 8; ++j)
                            dst[j] = make_float4(__uint_as_float(v[4 * j]), __uint_as_float(v[4 * j + 1]),
                                                 __uint_as_float(v[4 * j + 2]), __uint_as_float(v[4 * j + 3]));
                    }
                } else {
                    // rows >= d_out and columns past the bias column are exactly zero
                    float s = 0.f;
#pragma unroll
                    for (int j = 0; j < 32; ++j) { const float x = __uint_as_float(v[j]); s = fmaf(x, x, s); }
                    s = warp_sum(s);
                    if (lane == 0) { if (za > 32) atomicAdd(p.sq + item, s); else p.sq[item] = s; }
                }
            }
            tc_fence_before_sync();
            __syncwarp();
            if (lane == 0) mbar_arrive(&acc_empty[buf]);
        }
    } else if (warp >= 2 + EPI_WARPS) {
        // ------------------------------------------------ convert: pair f takes the chunks f, f + 6, ... of the CTA's
        // chunk sequence (all items strung together) into its own stage slot; warp h of the pair rows 32 h .. 32 h + 31
        const int f = (warp - (2 + EPI_WARPS)) >> 1, h = (warp - (2 + EPI_WARPS)) & 1;
        constexpr int HB = BK / 2;                             // rows per warp
        const int kbase = h * HB;
        const bool z_vec = (za & 7) == 0;
        const int vpr = za >> 3;                               // vectors per Zb row (z_vec)
        const int vshift = (vpr & (vpr - 1)) == 0 ? 31 - __clz(vpr | 1) : -1;     // log2 when a power of two
        uint8_t* zt = smem + f * STAGE_BYTES;
        uint8_t* at = zt + Z_BYTES;
        const uint32_t a_unit = lane >> 3, a_sub = (lane & 7) << 1;
        int seq = 0;                                           // chunks before the current item
        uint32_t my_phase = 0;
        bool ok = true;
        [[maybe_unused]] int tr = 0;
        for (int item = item0; item < n_items && ok; item += item_step) {
            long r0, r1; item_rows(item, r0, r1);
            const int nkb = (int)((r1 - r0 + BK - 1) / BK);
            int kb = (f - seq) % CONV_PAIRS; if (kb < 0) kb += CONV_PAIRS;
            for (; kb < nkb; kb += CONV_PAIRS) {
                const int g = seq + kb;                        // position in the CTA's chunk sequence
                const int rslot = g % n_raw; const uint32_t rphase = (uint32_t)((g / n_raw) & 1);
                const long rb = r0 + (long)kb * BK;
                const int nr = (int)min((long)BK, r1 - rb);
                // clip factors of the chunk's rows: example of its first row, then at most a few steps
                int e0 = 0, rem0 = 0;
                if (GRAD && p.clip) { e0 = (int)(rb / p.T); rem0 = (int)(rb - (long)e0 * p.T); }
                auto factor = [&](int k) {
                    int e = e0, r = rem0 + k;
                    while (r >= p.T) { r -= p.T; ++e; }
                    return __ldg(p.clip + e);
                };
                ok = mbar_wait(&raw_full[rslot], rphase, abort_flag, p.status);
                if (ok) ok = mbar_wait(&empty[f], my_phase ^ 1, abort_flag, p.status);
                if (!ok) break;
                my_phase ^= 1;
                if (f == 0 && h == 0 && lane == 0) { DPCLIP_TRACE_AT(1, tr); ++tr; }
                const uint8_t* ra = raw + rslot * chunk_bytes;
                const uint8_t* rz = ra + a_chunk;
                // ---- [A|1]: lane = column; element (k, lane) -> byte k * 128 + (((lane >> 3) ^ (k & 7)) << 4) + (lane & 7) * 2
                if (lane < aa) {
                    const unsigned short* src = reinterpret_cast<const unsigned short*>(ra) + lane + kbase * aa;
                    uint8_t* dst = at + kbase * 128;
                    if (nr == BK) {
                        // sixteen loads, then sixteen stores: a store after every load would wait for it (the
                        // compiler cannot tell the raw ring from the operand tile)
#pragma unroll
                        for (int k0 = 0; k0 < HB; k0 += 16) {
                            unsigned short v[16];
#pragma unroll
                            for (int j = 0; j < 16; ++j) v[j] = src[(k0 + j) * aa];
#pragma unroll
                            for (int j = 0; j < 16; ++j)
                                *reinterpret_cast<unsigned short*>(dst + (k0 + j) * 128 + (((a_unit ^ ((k0 + j) & 7)) << 4) | a_sub)) = v[j];
                        }
                    } else {
                        for (int k = 0; k < HB && kbase + k < nr; ++k)
                            *reinterpret_cast<unsigned short*>(dst + k * 128 + (((a_unit ^ (k & 7)) << 4) | a_sub)) = src[k * aa];
                    }
                }
                // ---- Zb: rows past the end of the item are stored as zeros
                if (z_vec) {
                    const int nv = (kbase + HB) * vpr, nvalid = nr * vpr;
                    for (int v0 = kbase * vpr + lane; v0 < nv; v0 += 128) {         // four vectors per lane at a time
                        uint4 w[4];
#pragma unroll
                        for (int u = 0; u < 4; ++u) {
                            const int v = v0 + 32 * u;
                            w[u] = v < nvalid ? *reinterpret_cast<const uint4*>(rz + v * 16) : make_uint4(0, 0, 0, 0);
                        }
#pragma unroll
                        for (int u = 0; u < 4; ++u) {
                            const int v = v0 + 32 * u;
                            if (v >= nv) continue;
                            int k, c;
                            if (vshift >= 0) { k = v >> vshift; c = (v & (vpr - 1)) << 3; }
                            else { k = v / vpr; c = (v - k * vpr) << 3; }
                            if (GRAD && p.clip && v < nvalid) {
                                const float cf = factor(k);
                                if (cf != 1.0f) {
                                    uint32_t* ww = reinterpret_cast<uint32_t*>(&w[u]);
#pragma unroll
                                    for (int j = 0; j < 4; ++j) {
                                        const __nv_bfloat162 h = __floats2bfloat162_rn(__uint_as_float(ww[j] << 16) * cf,
                                                                                        __uint_as_float(ww[j] & 0xFFFF0000u) * cf);
                                        ww[j] = *reinterpret_cast<const uint32_t*>(&h);
                                    }
                                }
                            }
                            *reinterpret_cast<uint4*>(zt + mn_off(k, c)) = w[u];
                        }
                    }
                } else {
                    const __nv_bfloat16* zsrc = reinterpret_cast<const __nv_bfloat16*>(rz);
                    for (int idx = kbase * za + lane; idx < (kbase + HB) * za; idx += 32) {
                        const int k = idx / za, c = idx - k * za;
                        float x = k < nr ? to_f32(zsrc[idx]) : 0.f;
                        if (GRAD && p.clip && k < nr) x *= factor(k);
                        *reinterpret_cast<__nv_bfloat16*>(zt + mn_off(k, c)) = __float2bfloat16_rn(x);
                    }
                }
                fence_proxy_async_smem();
                __syncwarp();
                if (lane == 0) { mbar_arrive(&full[f]); mbar_arrive(&raw_empty[rslot]); }
                if (f == 0 && h == 0 && lane == 0) { DPCLIP_TRACE_AT(1, tr); ++tr; }
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
    if (warp == 1) { tc_fence_after_sync(); tmem_dealloc(tmem_base, 2 * ACC_COLS); }
}

}  // namespace tc
}  // namespace dpclip
