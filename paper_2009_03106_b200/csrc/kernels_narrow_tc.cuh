// Narrow layers on the tensor cores (bf16): d_in (+1 with a bias) <= 32, d_out <= 64, dense rows --
// e.g. the first 3x3 convolution of an RGB network (d_in = 27, T = H*W large).
//
// The fp32-ALU streaming kernels (kernels_narrow.cuh) spend ~40 issue slots and 12-33 cycles of the
// shared-memory pipe per input row and warp; with one example (or row slice) per SM that is 17-20 us for
// the 1024 rows of a 32 x 32 image, whatever the memory system does.  The contraction itself is tiny, so
// here it goes to the tensor cores and the SM's threads only MOVE data: rows of 54 bytes cannot be fetched
// by TMA, so fifteen fill warps load 32-row blocks (contiguous in memory, 128-bit loads, one block per warp
// in registers at a time = fifteen blocks in flight per SM) and scatter them into shared memory in the
// MN-major 128-byte-swizzled operand layout:
//     Zb tile   M = 128 (d_out real columns, the rest stays zero), 32 rows (K) per stage
//     [A|1] tile N = 64 (d_in real columns, then the all-ones bias column, the rest stays zero)
// One thread issues two 128 x 64 x 16 MMAs per stage into a 64-column accumulator in tensor memory.
//   NORM: one item per example; the epilogue squares and sums the 64 x 32 block that holds the example's
//         gradient (the padding is exactly zero), so the per-example gradient never leaves the SM.
//   GRAD: one row slice per CTA, Zb scaled by the example's clip factor on its way to shared memory (fp32
//         product, one rounding to bf16); the tile goes to the partial buffer that narrow_reduce_kernel sums.
// Every wait is bounded; on a timeout the CTA sets the status word and unwinds.
#pragma once
#include "tc_common.cuh"

namespace dpclip {
namespace tc {
namespace ntc {
constexpr int BK = 32;                           // rows per stage
constexpr int Z_BYTES = 2 * BK * 128;            // two 64-column chunks (the second one all zero)
constexpr int A_BYTES = BK * 128;
constexpr int STAGE_BYTES = Z_BYTES + A_BYTES;   // 12 KB
constexpr int FILL_WARPS = 15, EPI_WARPS = 4;   // 20 warps in all: 96 registers per thread
// Every fill warp owns one shared-memory slot (stage g of the CTA's sequence lives in slot g % 15 and is
// filled by warp g % 15), so a slot's barrier phases are seen by one producer in order.
constexpr int STAGES = FILL_WARPS;
constexpr int THREADS = 32 * (1 + EPI_WARPS + FILL_WARPS);     // warp 0 MMA, warps 1..4 epilogue, 5..19 fill
constexpr int SMEM_BYTES = STAGES * STAGE_BYTES + 256 + 1024;
constexpr int ACC_COLS = 64;                     // accumulator columns per buffer (N)

struct Params {
    const __nv_bfloat16* A; const __nv_bfloat16* Z;    // dense rows: row r at A + r * d_in, Z + r * d_out
    int T, d_in, d_out, has_bias;
    int n_items;                       // NORM: examples
    long rows_total, rows_per_cta;     // GRAD: one slice per CTA (rows_per_cta a multiple of BK)
    int vec;                           // every stage starts on a 16-byte boundary in both inputs
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
}  // namespace ntc

template <bool GRAD>
__global__ void __launch_bounds__(ntc::THREADS, 1)
narrow_tc_kernel(const ntc::Params p) {
    using namespace ntc;
    extern __shared__ uint8_t smem_raw[];
    uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
    uint64_t* full = reinterpret_cast<uint64_t*>(smem + STAGES * STAGE_BYTES);
    uint64_t* empty = full + STAGES;
    uint64_t* acc_full = empty + STAGES;
    uint64_t* acc_empty = acc_full + 2;
    uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(acc_empty + 2);
    volatile int* abort_flag = reinterpret_cast<volatile int*>(tmem_slot + 1);

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    if (threadIdx.x == 0) DPCLIP_TRACE_AT(0, 254);
    // operand tiles start all zero; the fill warps only ever write the real columns, so the padding stays
    // zero for the whole kernel.  The bias column of [A|1] is set once.
    for (int i = threadIdx.x; i < STAGES * STAGE_BYTES / 16; i += THREADS)
        reinterpret_cast<uint4*>(smem)[i] = make_uint4(0, 0, 0, 0);
    __syncthreads();
    if (p.has_bias)
        for (int i = threadIdx.x; i < STAGES * BK; i += THREADS) {
            const int s = i / BK, k = i - s * BK;
            *reinterpret_cast<__nv_bfloat16*>(smem + s * STAGE_BYTES + Z_BYTES + mn_off(k, p.d_in)) = __float2bfloat16_rn(1.f);
        }
    if (threadIdx.x == 0) {
        for (int s = 0; s < STAGES; ++s) { mbar_init(&full[s], 1); mbar_init(&empty[s], 1); }
        for (int b = 0; b < 2; ++b) { mbar_init(&acc_full[b], 1); mbar_init(&acc_empty[b], EPI_WARPS); }
        *abort_flag = 0;
        mbar_fence_init();
    }
    if (warp == 0) { tmem_alloc(tmem_slot, 2 * ACC_COLS); tmem_relinquish(); }
    fence_proxy_async_smem();
    tc_fence_before_sync();
    __syncthreads();
    tc_fence_after_sync();
    const uint32_t tmem_base = *tmem_slot;

    // items of this CTA: NORM = examples blockIdx.x, + gridDim.x, ...; GRAD = its one row slice
    const int n_items = GRAD ? 1 : p.n_items;
    const int item0 = GRAD ? 0 : blockIdx.x, item_step = GRAD ? 1 : gridDim.x;
    auto item_rows = [&](int item, long& r0, long& r1) {
        if (GRAD) { r0 = (long)blockIdx.x * p.rows_per_cta; r1 = min(r0 + p.rows_per_cta, p.rows_total); }
        else { r0 = (long)item * p.T; r1 = r0 + p.T; }
    };

    if (warp == 0) {
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
                        // MN-major, 128-byte swizzle: 64-column chunks BK * 128 bytes apart, 8-row groups 1024
                        // bytes apart; 16 rows = 2048 bytes
                        const uint64_t dz = make_smem_desc_sw128(zb + k16 * 2048, BK * 128, 1024);
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
    } else if (warp <= EPI_WARPS) {
        // ------------------------------------------------ epilogue: warp w reads tensor-memory lanes 32 * (w % 4) ..
        const int quarter = warp & 3;
        int it = 0;
        for (int item = item0; item < n_items; item += item_step, ++it) {
            const int buf = it & 1; const uint32_t acc_phase = (it >> 1) & 1;
            if (!mbar_wait(&acc_full[buf], acc_phase, abort_flag, p.status)) break;
            if (threadIdx.x == 32 * EPI_WARPS) DPCLIP_TRACE_AT(3, it);
            tc_fence_after_sync();
            if (quarter * 32 < p.d_out) {                      // lanes of this quarter hold output rows m = 32 q + lane
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
                    if (lane == 0) { if (p.d_out > 32) atomicAdd(p.sq + item, s); else p.sq[item] = s; }
                }
            }
            tc_fence_before_sync();
            __syncwarp();
            if (lane == 0) mbar_arrive(&acc_empty[buf]);
        }
    } else {
        // ------------------------------------------------ fill: warp f takes the stages f, f + 15, ... of the CTA's
        // stage sequence (all items strung together), so fifteen blocks are in flight per SM.
        //   [A|1]: lane c copies column c of the block: its 32 loads (one per row, 2 bytes, consecutive lanes
        //          read consecutive elements) are issued first; the shared-memory offset of (row, c) is the row's
        //          compile-time part plus a per-lane part, so a copied element costs a few instructions.
        //   Zb:    rows of d_out = 8, 16, ..., 64 elements on 16-byte boundaries go as 128-bit vectors (one
        //          vector never leaves its row); anything else element by element.
        const int f = warp - (1 + EPI_WARPS);
        const int za = p.d_out, aa = p.d_in;
        const bool z_vec = p.vec && (za & 7) == 0;
        const int vpr = za >> 3;                               // vectors per Zb row (z_vec)
        const int vshift = (vpr & (vpr - 1)) == 0 ? 31 - __clz(vpr | 1) : -1;     // log2 when a power of two
        const int nvz_lane = z_vec ? (BK * vpr + 31) >> 5 : 0; // vectors per lane and stage
        int seq = 0;                                           // stages before the current item, modulo FILL_WARPS
        uint32_t my_phase = 0;                                 // this warp's slot (stage f) is used in order
        uint8_t* zt = smem + f * STAGE_BYTES;
        uint8_t* at = zt + Z_BYTES;
        bool ok = true;
        [[maybe_unused]] int tr = 0;
        if (f == 0 && lane == 0) DPCLIP_TRACE_AT(1, 255);
        for (int item = item0; item < n_items && ok; item += item_step) {
            long r0, r1; item_rows(item, r0, r1);
            const int nkb = (int)((r1 - r0 + BK - 1) / BK);
            int kb = f - seq; if (kb < 0) kb += FILL_WARPS;
            for (; kb < nkb; kb += FILL_WARPS) {
                const long rb = r0 + (long)kb * BK;
                const int nr = (int)min((long)BK, r1 - rb);
                const __nv_bfloat16* zsrc = p.Z + (size_t)rb * za;
                const unsigned short* asrc = reinterpret_cast<const unsigned short*>(p.A + (size_t)rb * aa) + lane;
                // ---- loads first, then the wait for the slot
                unsigned short av[BK];
                const bool a_lane = lane < aa;
                if (nr == BK) {
#pragma unroll
                    for (int k = 0; k < BK; ++k) av[k] = a_lane ? __ldg(asrc + k * aa) : (unsigned short)0;
                } else {
#pragma unroll
                    for (int k = 0; k < BK; ++k) av[k] = (a_lane && k < nr) ? __ldg(asrc + k * aa) : (unsigned short)0;
                }
                constexpr int NVZ = (BK * 64) / (8 * 32);      // Zb vectors per lane at d_out = 64
                uint4 vz[NVZ];
                const int nvalid = nr * vpr;
#pragma unroll
                for (int u = 0; u < NVZ; ++u) {
                    vz[u] = make_uint4(0, 0, 0, 0);            // rows past the end of the item are stored as zeros
                    if (u < nvz_lane) {
                        const int v = u * 32 + lane;
                        if (v < nvalid) vz[u] = __ldg(reinterpret_cast<const uint4*>(zsrc) + v);
                    }
                }
                // clip factors of the block's rows: example of its first row, then at most a few steps
                int e0 = 0, rem0 = 0;
                if (GRAD && p.clip) { e0 = (int)(rb / p.T); rem0 = (int)(rb - (long)e0 * p.T); }
                auto factor = [&](int k) {
                    int e = e0, r = rem0 + k;
                    while (r >= p.T) { r -= p.T; ++e; }
                    return __ldg(p.clip + e);
                };
                if (f == 0 && lane == 0) { DPCLIP_TRACE_AT(1, tr); ++tr; }
                ok = mbar_wait(&empty[f], my_phase ^ 1, abort_flag, p.status);
                if (!ok) break;
                my_phase ^= 1;
                // ---- [A|1]: element (k, lane) -> byte k * 128 + (((lane >> 3) ^ (k & 7)) << 4) + (lane & 7) * 2
                if (a_lane) {
                    const uint32_t unit = lane >> 3, sub = (lane & 7) << 1;
#pragma unroll
                    for (int k = 0; k < BK; ++k)
                        if (k < nr) *reinterpret_cast<unsigned short*>(at + k * 128 + (((unit ^ (k & 7)) << 4) | sub)) = av[k];
                }
                // ---- Zb
                if (z_vec) {
#pragma unroll
                    for (int u = 0; u < NVZ; ++u) {
                        if (u >= nvz_lane) break;
                        const int v = u * 32 + lane;
                        if (v >= BK * vpr) continue;
                        int k, c;
                        if (vshift >= 0) { k = v >> vshift; c = (v & (vpr - 1)) << 3; }
                        else { k = v / vpr; c = (v - k * vpr) << 3; }
                        uint4 w = vz[u];
                        if (GRAD && p.clip && k < nr) {
                            const float cf = factor(k);
                            if (cf != 1.0f) {
                                uint32_t* ww = reinterpret_cast<uint32_t*>(&w);
#pragma unroll
                                for (int j = 0; j < 4; ++j) {
                                    const __nv_bfloat162 h = __floats2bfloat162_rn(__uint_as_float(ww[j] << 16) * cf,
                                                                                    __uint_as_float(ww[j] & 0xFFFF0000u) * cf);
                                    ww[j] = *reinterpret_cast<const uint32_t*>(&h);
                                }
                            }
                        }
                        *reinterpret_cast<uint4*>(zt + mn_off(k, c)) = w;
                    }
                } else {
                    for (int idx = lane; idx < BK * za; idx += 32) {
                        const int k = idx / za, c = idx - k * za;
                        float x = k < nr ? to_f32(zsrc[idx]) : 0.f;
                        if (GRAD && p.clip && k < nr) x *= factor(k);
                        *reinterpret_cast<__nv_bfloat16*>(zt + mn_off(k, c)) = __float2bfloat16_rn(x);
                    }
                }
                fence_proxy_async_smem();
                __syncwarp();
                if (lane == 0) mbar_arrive(&full[f]);
                if (f == 0 && lane == 0) { DPCLIP_TRACE_AT(1, tr); ++tr; }
            }
            seq = (seq + nkb) % FILL_WARPS;
        }
    }

    // ---------------------------------------------------- teardown
    if (*abort_flag) {
        for (int i = 0; i < 64; ++i) __nanosleep(1000);
    }
    tc_fence_before_sync();
    __syncthreads();
    if (warp == 0) { tc_fence_after_sync(); tmem_dealloc(tmem_base, 2 * ACC_COLS); }
}

}  // namespace tc
}  // namespace dpclip
