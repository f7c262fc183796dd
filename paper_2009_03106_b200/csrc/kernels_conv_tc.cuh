// Convolution layers from their INPUT feature map on the tensor cores (bf16, implicit im2col).
//
// Algorithm 3 of the paper unfolds the input into a patch matrix (k_h * k_w copies of every pixel) and
// multiplies; here the patch matrix exists only as 64-row operand tiles in shared memory:
//   * one thread copies each example's feature map (C * H * W bf16, contiguous) into one of two raw buffers
//     in shared memory with an untiled bulk copy, and fetches the matching 64-row tiles of Zb by TMA straight
//     into the MN-major operand layout;
//   * eight converter warps build the patch tile of the stage in the K-MAJOR operand layout (N-row = patch
//     column n = (c, ky, kx), 64 contraction rows t = 128 contiguous bytes); eight consecutive t share their
//     output row y', so one 16-byte unit of the tile is eight neighbouring pixels of one input row (zero
//     outside the map); the all-ones bias column is N-row d_in;
//   * GRAD only: four warps scale the Zb tile in place by the example's clip factor (one rounding to bf16);
//   * one thread issues four 128 x N x 16 MMAs per stage (A operand MN-major, B operand K-major) into one of
//     two 256-column accumulators in tensor memory; four epilogue warps.
//   NORM: item = (example, block of 256 patch columns); the epilogue squares and sums the block -> sq[i] (atomics).
//   GRAD: item = (slice of examples, block of 256 patch columns); the tile goes to the partial buffer that
//         reduce_partials_kernel sums (the bias gradient is column d_in of the last block).
// Zb may be [B][T][d_out] or [B][d_out][T] (then its tiles are K-major too).
// Restrictions (checked on the host; anything else takes the fp32-ALU kernel): stride 1, output width 8, 16, 32
// or 64, T a multiple of 64, d_out a multiple of 8 and at most 128, feature map at most 32 KB per example.
// Every wait is bounded; on a timeout the CTA sets the status word and unwinds.
#pragma once
#include "tc_common.cuh"

namespace dpclip {
namespace tc {
namespace ctc {
constexpr int BK = 64;                           // contraction rows (t) per stage
constexpr int BN = 256;                          // patch columns per item
constexpr int Z_BYTES = 2 * BK * 128;            // Zb tile: two 64-column chunks
constexpr int P_BYTES = BN * 128;                // patch tile: 256 N-rows x 64 t
constexpr int STAGE_BYTES = Z_BYTES + P_BYTES;   // 48 KB
constexpr int STAGES = 3;
constexpr int X_BYTES = 32 * 1024;               // raw feature map of one example (two buffers)
constexpr int PATCH_WARPS = 16, SCALE_WARPS = 4, EPI_WARPS = 4;   // the converter is bound by the latency of its
                                                                  // dependent integer chains: four warps per scheduler
constexpr int THREADS = 32 * (2 + EPI_WARPS + PATCH_WARPS + SCALE_WARPS);   // warp 0 copies, 1 MMA, 2..5 epilogue, 6..21 patches, 22..25 scale
constexpr int TAB_BYTES = 2 * BN * 8;             // patch-column tables of two items in flight
constexpr int SMEM_BYTES = STAGES * STAGE_BYTES + 2 * X_BYTES + TAB_BYTES + 256 + 1024;

struct Params {
    const __nv_bfloat16* X;            // [B][C][H][W]
    int B, C, H, W, kh, kw, pad, Ho, Wo, wo_shift;
    int T, d_in, d_out, has_bias;
    int z_cm;                          // Zb is [B][d_out][T] (the layout of dL/dZ itself): its tiles are K-major
    int tiles_n;                       // blocks of 256 patch columns (d_in + bias columns in all)
    int n_items;                       // NORM: B * tiles_n; GRAD: slices * tiles_n
    int ex_per_item;                   // GRAD: examples per slice (NORM: 1)
    const float* clip;                 // GRAD: [B] or NULL
    float* sq;                         // NORM: [B], pre-zeroed
    float* part;                       // GRAD: [n_items][128][256] partial tiles
    int* status;
};
// Eight consecutive bf16 starting dx elements into `cur` (|dx| <= 3), spilling into the neighbouring vector `nb`
// (the one before `cur` when dx < 0, the one after it when dx > 0).  Branch-free: lanes of a warp hold different dx.
__device__ __forceinline__ uint4 shifted8(const uint4& cur, const uint4& nb, int dx) {
    const bool neg = dx < 0;
    const int half = dx & 1;                       // odd shifts move by 16 bits inside the words
    const int wsh = (dx - half) >> 1;              // whole 32-bit words: -2 .. 1
    const bool one = neg ? wsh == -1 : wsh == 1;   // second position of the six-word window
    // window of six words that holds the result for both positions
    const uint32_t l0 = neg ? nb.z : cur.x, l1 = neg ? nb.w : cur.y, l2 = neg ? cur.x : cur.z,
                   l3 = neg ? cur.y : cur.w, l4 = neg ? cur.z : nb.x, l5 = neg ? cur.w : nb.y;
    const uint32_t w0 = one ? l1 : l0, w1 = one ? l2 : l1, w2 = one ? l3 : l2, w3 = one ? l4 : l3, w4 = one ? l5 : l4;
    const uint32_t sh = (uint32_t)half * 16u;
    return make_uint4(__funnelshift_r(w0, w1, sh), __funnelshift_r(w1, w2, sh), __funnelshift_r(w2, w3, sh),
                      __funnelshift_r(w3, w4, sh));
}
// The same for a dx that is uniform across the warp: a plain switch.
__device__ __forceinline__ uint4 shifted8u(const uint4& prev, const uint4& cur, const uint4& next, int dx) {
    switch (dx) {
        case -3: return make_uint4(__funnelshift_r(prev.z, prev.w, 16), __funnelshift_r(prev.w, cur.x, 16),
                                   __funnelshift_r(cur.x, cur.y, 16), __funnelshift_r(cur.y, cur.z, 16));
        case -2: return make_uint4(prev.w, cur.x, cur.y, cur.z);
        case -1: return make_uint4(__funnelshift_r(prev.w, cur.x, 16), __funnelshift_r(cur.x, cur.y, 16),
                                   __funnelshift_r(cur.y, cur.z, 16), __funnelshift_r(cur.z, cur.w, 16));
        case 1:  return make_uint4(__funnelshift_r(cur.x, cur.y, 16), __funnelshift_r(cur.y, cur.z, 16),
                                   __funnelshift_r(cur.z, cur.w, 16), __funnelshift_r(cur.w, next.x, 16));
        case 2:  return make_uint4(cur.y, cur.z, cur.w, next.x);
        case 3:  return make_uint4(__funnelshift_r(cur.y, cur.z, 16), __funnelshift_r(cur.z, cur.w, 16),
                                   __funnelshift_r(cur.w, next.x, 16), __funnelshift_r(next.x, next.y, 16));
        default: return cur;
    }
}
}  // namespace ctc

template <bool GRAD>
__global__ void __launch_bounds__(ctc::THREADS, 1)
conv_tc_kernel(const __grid_constant__ CUtensorMap map_z, const ctc::Params p) {
    using namespace ctc;
    extern __shared__ uint8_t smem_raw[];
    uint8_t* smem = smem_raw + ((1024u - (smem_u32(smem_raw) & 1023u)) & 1023u);
    uint8_t* xraw = smem + STAGES * STAGE_BYTES;
    int2* col_tab = reinterpret_cast<int2*>(xraw + 2 * X_BYTES);          // per patch column: channel offset, dy | dx | kind
    uint64_t* zfull = reinterpret_cast<uint64_t*>(xraw + 2 * X_BYTES + TAB_BYTES);    // Zb tile landed
    uint64_t* ready = zfull + STAGES;                                      // patch tile built (and Zb scaled)
    uint64_t* empty = ready + STAGES;                                      // MMAs done with the stage
    uint64_t* xfull = empty + STAGES;                                      // feature map landed
    uint64_t* xempty = xfull + 2;                                          // patch warps done with it
    uint64_t* acc_full = xempty + 2;
    uint64_t* acc_empty = acc_full + 2;
    uint64_t* tab_full = acc_empty + 2;                                    // column table of an item written (two in flight)
    uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(tab_full + 2);
    volatile int* abort_flag = reinterpret_cast<volatile int*>(tmem_slot + 1);

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    if (threadIdx.x == 0) {
        DPCLIP_TRACE_AT(0, 254);
        for (int s = 0; s < STAGES; ++s) {
            mbar_init(&zfull[s], 1);
            mbar_init(&ready[s], PATCH_WARPS + (GRAD ? SCALE_WARPS : 0));
            mbar_init(&empty[s], 1);
        }
        for (int b = 0; b < 2; ++b) {
            mbar_init(&xfull[b], 1); mbar_init(&xempty[b], PATCH_WARPS);
            mbar_init(&acc_full[b], 1); mbar_init(&acc_empty[b], EPI_WARPS);
            mbar_init(&tab_full[b], PATCH_WARPS);
        }
        *abort_flag = 0;
        mbar_fence_init();
        tma_prefetch_desc(&map_z);
    }
    if (warp == 1) { tmem_alloc(tmem_slot, 512); tmem_relinquish(); }
    tc_fence_before_sync();
    __syncthreads();
    tc_fence_after_sync();
    const uint32_t tmem_base = *tmem_slot;

    const int nkb = p.T / BK;                               // stages per example
    const int x_bytes = p.C * p.H * p.W * 2;
    const int z_chunks = (p.d_out + 63) >> 6;               // 64-column chunks of Zb that hold data
    // item -> (first example, number of examples, block of patch columns)
    auto decode = [&](int item, int& e0, int& ne, int& j) {
        const int outer = item / p.tiles_n;
        j = item - outer * p.tiles_n;
        e0 = outer * p.ex_per_item;
        ne = min(p.ex_per_item, p.B - e0);
    };

    if (warp == 0) {
        // ------------------------------------------------ copies: feature maps (bulk) and Zb tiles (TMA)
        if (lane == 0) {
            int g = 0, xe = 0;
            bool ok = true;
            for (int item = blockIdx.x; item < p.n_items && ok; item += gridDim.x) {
                int e0, ne, j; decode(item, e0, ne, j);
                for (int e = e0; e < e0 + ne && ok; ++e, ++xe) {
                    const int b = xe & 1;
                    ok = mbar_wait(&xempty[b], ((xe >> 1) & 1) ^ 1, abort_flag, p.status);
                    if (!ok) break;
                    mbar_arrive_expect_tx(&xfull[b], (uint32_t)x_bytes);
                    asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];"
                                 ::"r"(smem_u32(xraw + b * X_BYTES)), "l"(p.X + (size_t)e * p.C * p.H * p.W),
                                   "r"((uint32_t)x_bytes), "r"(smem_u32(&xfull[b])) : "memory");
                    for (int kb = 0; kb < nkb; ++kb, ++g) {
                        const int s = g % STAGES;
                        ok = mbar_wait(&empty[s], ((g / STAGES) & 1) ^ 1, abort_flag, p.status);
                        if (!ok) break;
                        uint8_t* zt = smem + s * STAGE_BYTES;
                        if (p.z_cm) {
                            // [d_out rows][64 t]: one box, 128 bytes per row (rows past d_out keep stale values: they
                            // only feed accumulator rows nobody reads)
                            mbar_arrive_expect_tx(&zfull[s], (uint32_t)(p.d_out * 128));
                            tma_load_2d(zt, &map_z, &zfull[s], kb * BK, e * p.d_out);
                        } else {
                            mbar_arrive_expect_tx(&zfull[s], (uint32_t)(z_chunks * BK * 128));
                            for (int c = 0; c < z_chunks; ++c)
                                tma_load_2d(zt + c * (BK * 128), &map_z, &zfull[s], c * 64, e * p.T + kb * BK);
                        }
                    }
                }
            }
        }
    } else if (warp == 1) {
        // ------------------------------------------------ MMA issuer
        if (lane == 0) {
            int g = 0, it = 0;
            bool ok = true;
            DPCLIP_TRACE_AT(0, 255);
            for (int item = blockIdx.x; item < p.n_items && ok; item += gridDim.x, ++it) {
                int e0, ne, j; decode(item, e0, ne, j);
                const int n_cols = min(BN, p.d_in + p.has_bias - j * BN);
                // N in steps of 32: the epilogue reads the accumulator 32 columns at a time, and patch rows past the
                // last real column are zero
                const uint32_t idesc = make_idesc_bf16(128, (n_cols + 31) & ~31, p.z_cm ? 0 : 1, 0);
                const int buf = it & 1;
                ok = mbar_wait(&acc_empty[buf], ((it >> 1) & 1) ^ 1, abort_flag, p.status);
                if (!ok) break;
                tc_fence_after_sync();
                for (int kk = 0; kk < ne * nkb; ++kk, ++g) {
                    const int s = g % STAGES; const uint32_t ph = (g / STAGES) & 1;
                    ok = mbar_wait(&zfull[s], ph, abort_flag, p.status);
                    if (ok) ok = mbar_wait(&ready[s], ph, abort_flag, p.status);
                    if (!ok) break;
                    DPCLIP_TRACE_AT(2, g);
                    tc_fence_after_sync();
                    const uint32_t zb = smem_u32(smem + s * STAGE_BYTES), pb = zb + Z_BYTES;
#pragma unroll
                    for (int k16 = 0; k16 < BK / 16; ++k16) {
                        // Zb: MN-major, 64-column chunks BK * 128 bytes apart (stride 0 when only one holds data:
                        // the M rows 64..127 then re-read it and are never used); 16 rows = 2048 bytes.
                        // patches: K-major, 8-row groups 1024 bytes apart; 16 contraction elements = 32 bytes.
                        const uint64_t dz = p.z_cm ? make_smem_desc_sw128(zb + k16 * 32, 16, 1024)      // K-major rows of 64 t
                                                   : make_smem_desc_sw128(zb + k16 * 2048, z_chunks > 1 ? BK * 128 : 0, 1024);
                        const uint64_t dp = make_smem_desc_sw128(pb + k16 * 32, 16, 1024);
                        mma_bf16_ss(tmem_base + buf * BN, dz, dp, idesc, (kk == 0 && k16 == 0) ? 0u : 1u);
                    }
                    mma_commit(&empty[s]);
                }
                if (!ok) break;
                mma_commit(&acc_full[buf]);
            }
        }
    } else if (warp < 2 + EPI_WARPS) {
        // ------------------------------------------------ epilogue: warp w reads tensor-memory lanes 32 * (w % 4) ..
        const int quarter = warp & 3;
        const int m = quarter * 32 + lane;                     // output row (d_out index) of this thread
        int it = 0;
        for (int item = blockIdx.x; item < p.n_items; item += gridDim.x, ++it) {
            int e0, ne, j; decode(item, e0, ne, j);
            const int n_cols = min(BN, p.d_in + p.has_bias - j * BN);
            const int buf = it & 1;
            if (!mbar_wait(&acc_full[buf], (it >> 1) & 1, abort_flag, p.status)) break;
            if (threadIdx.x == 64) DPCLIP_TRACE_AT(3, 2 * it);
            tc_fence_after_sync();
            float s = 0.f;
            if (quarter * 32 < p.d_out) {
                const uint32_t t_row = tmem_base + ((uint32_t)(quarter * 32) << 16) + buf * BN;
#pragma unroll 1
                for (int c0 = 0; c0 < n_cols; c0 += 32) {
                    uint32_t v[32];
                    tmem_ld_32x32(t_row + c0, v);
                    tmem_ld_wait();
                    if (GRAD) {
                        if (m < p.d_out) {
                            float4* dst = reinterpret_cast<float4*>(p.part + ((size_t)item * 128 + m) * BN + c0);
#pragma unroll
                            for (int q = 0; q < 8; ++q)
                                dst[q] = make_float4(__uint_as_float(v[4 * q]), __uint_as_float(v[4 * q + 1]),
                                                     __uint_as_float(v[4 * q + 2]), __uint_as_float(v[4 * q + 3]));
                        }
                    } else if (m < p.d_out) {
                        // patch columns past the last real one are exactly zero
#pragma unroll
                        for (int q = 0; q < 32; ++q) { const float x = __uint_as_float(v[q]); s = fmaf(x, x, s); }
                    }
                }
            }
            tc_fence_before_sync();
            __syncwarp();
            if (lane == 0) mbar_arrive(&acc_empty[buf]);
            if (threadIdx.x == 64) DPCLIP_TRACE_AT(3, 2 * it + 1);
            if (!GRAD && quarter * 32 < p.d_out) {
                s = warp_sum(s);
                if (lane == 0) atomicAdd(p.sq + e0, s);
            }
        }
    } else if (warp < 2 + EPI_WARPS + PATCH_WARPS) {
        // ------------------------------------------------ patch tiles.  The k_w patch columns (c, ky, 0 .. k_w - 1) read
        // the same input row shifted by one pixel each, so a thread takes one such GROUP of columns and one
        // K-unit u (eight consecutive t = one output row y', eight neighbouring x'): it loads the aligned 16-byte
        // vector of the row and its two neighbours once, and every column of the group is a funnel shift of
        // them (zeros at the edge of the map), stored as the 16-byte unit u of that column's N-row.  Lanes =
        // (u = t % 8, group t / 8): the eight u of a group read 128 contiguous bytes and write 128 contiguous
        // bytes per column.  Per unit ~10 instructions; with one thread per unit and column the converter
        // needed ~45 and bounded the kernel (issue slots: 0.6 us per stage before a single load).
        const int t = threadIdx.x - 32 * (2 + EPI_WARPS);      // 0 .. 511
        constexpr int GQ = 4 * PATCH_WARPS;                    // groups per pass
        const int u = t & 7, gq = t >> 3;
        const bool vec_rows = (p.W & 7) == 0 && p.pad <= 3 && p.kw - 1 - p.pad <= 3;
        const bool fast3 = vec_rows && p.kw == 3 && p.pad == 1;
        int g = 0, xe = 0, it = 0;
        bool ok = true;
        for (int item = blockIdx.x; item < p.n_items && ok; item += gridDim.x, ++it) {
            int e0, ne, j; decode(item, e0, ne, j);
            const int n0 = j * BN;                                         // first patch column of the block
            const int n_real = min(BN, p.d_in - n0);                       // real columns in the block (> 0)
            const int n_rows = (min(BN, p.d_in + p.has_bias - n0) + 31) & ~31;     // N-rows the MMAs read
            const int rg0 = n0 / p.kw;                                     // first group that overlaps the block
            const int n_groups = (n0 + n_real - 1) / p.kw - rg0 + 1;
            // The item's groups, decoded once: thread t writes the entry of group t.  Two tables (item parity):
            // nobody can still be reading the one written here, because the table of the item before this one
            // was complete only after every warp had finished the item before that.
            int2* tab = col_tab + (it & 1) * BN;
            {
                if (t < n_groups) {
                    const int rg = rg0 + t, c = rg / p.kh, ky = rg - c * p.kh;
                    tab[t] = make_int2(c * p.H * p.W, ky - p.pad);
                }
                __syncwarp();
                if (lane == 0) mbar_arrive(&tab_full[it & 1]);
                ok = mbar_wait(&tab_full[it & 1], (it >> 1) & 1, abort_flag, p.status);
                if (!ok) break;
            }
            // 3 x 3 kernels with one pixel of padding (the common case): everything that does not depend on the
            // stage is worked out here, for the at most two groups a thread owns (86 groups per block of 256
            // columns, 64 groups per pass): byte offset of the channel, ky - pad, and for each of the three columns
            // whether it lies in this block and where its 16-byte unit goes in the tile.
            int f_coff[2] = {0, 0}, f_dy[2] = {0, 0};
            uint32_t f_soff[2][3];
            bool f_ok[2][3];
#pragma unroll
            for (int gs = 0; gs < 2; ++gs) {
                const int gi = gq + GQ * gs, rg = rg0 + gi, c = rg / p.kh;
                f_coff[gs] = c * p.H * p.W * 2; f_dy[gs] = rg - c * p.kh - p.pad;
#pragma unroll
                for (int kx = 0; kx < 3; ++kx) {
                    const int n = rg * 3 + kx - n0;
                    f_ok[gs][kx] = fast3 && gi < n_groups && (unsigned)n < (unsigned)n_real;
                    f_soff[gs][kx] = (uint32_t)(n * 128) + (((uint32_t)u ^ (uint32_t)(n & 7)) << 4);
                }
            }
            for (int e = e0; e < e0 + ne && ok; ++e, ++xe) {
                const int b = xe & 1;
                ok = mbar_wait(&xfull[b], (xe >> 1) & 1, abort_flag, p.status);
                if (!ok) break;
                if (t == 0) DPCLIP_TRACE_AT(1, 128 + xe);
                const unsigned short* xs = reinterpret_cast<const unsigned short*>(xraw + b * X_BYTES);
                for (int kb = 0; kb < nkb; ++kb, ++g) {
                    const int s = g % STAGES;
                    ok = mbar_wait(&empty[s], ((g / STAGES) & 1) ^ 1, abort_flag, p.status);
                    if (!ok) break;
                    if (t == 0) DPCLIP_TRACE_AT(1, 2 * g);
                    uint8_t* pt = smem + s * STAGE_BYTES + Z_BYTES;
                    const int t0 = kb * BK + 8 * u;
                    const int yb = t0 >> p.wo_shift, xb = t0 & (p.Wo - 1);
                    const uint4 zero = make_uint4(0u, 0u, 0u, 0u);
                    if (fast3) {
                        const uint8_t* xb_ptr = reinterpret_cast<const uint8_t*>(xs) + (xb >> 3) * 16;
                        const bool has_prev = xb > 0, has_next = xb + 8 < p.W;
#pragma unroll
                        for (int gs = 0; gs < 2; ++gs) {
                            if (!(f_ok[gs][0] || f_ok[gs][1] || f_ok[gs][2])) continue;
                            const int y = yb + f_dy[gs];
                            const bool live = (unsigned)y < (unsigned)p.H;
                            const uint4* rowv = reinterpret_cast<const uint4*>(xb_ptr + f_coff[gs] + y * p.W * 2);
                            const uint4 cur = live ? rowv[0] : zero;
                            const uint4 prev = (live && has_prev) ? rowv[-1] : zero;
                            const uint4 next = (live && has_next) ? rowv[1] : zero;
                            if (f_ok[gs][0])
                                *reinterpret_cast<uint4*>(pt + f_soff[gs][0]) =
                                    make_uint4(__funnelshift_r(prev.w, cur.x, 16), __funnelshift_r(cur.x, cur.y, 16),
                                               __funnelshift_r(cur.y, cur.z, 16), __funnelshift_r(cur.z, cur.w, 16));
                            if (f_ok[gs][1]) *reinterpret_cast<uint4*>(pt + f_soff[gs][1]) = cur;
                            if (f_ok[gs][2])
                                *reinterpret_cast<uint4*>(pt + f_soff[gs][2]) =
                                    make_uint4(__funnelshift_r(cur.x, cur.y, 16), __funnelshift_r(cur.y, cur.z, 16),
                                               __funnelshift_r(cur.z, cur.w, 16), __funnelshift_r(cur.w, next.x, 16));
                        }
                    } else
                    for (int gi = gq; gi < n_groups; gi += GQ) {
                        const int2 grp = tab[gi];
                        const int y = yb + grp.y;
                        const bool live = (unsigned)y < (unsigned)p.H;
                        const unsigned short* row = xs + grp.x + y * p.W;
                        uint4 cur = zero, prev = zero, next = zero;
                        if (vec_rows && live) {
                            const uint4* rowv = reinterpret_cast<const uint4*>(row) + (xb >> 3);
                            cur = rowv[0];
                            if (xb > 0) prev = rowv[-1];
                            if (xb + 8 < p.W) next = rowv[1];
                        }
                        int n = (rg0 + gi) * p.kw - n0;                    // N-row of the group's first column
#pragma unroll 1
                        for (int kx = 0; kx < p.kw; ++kx, ++n) {
                            if ((unsigned)n >= (unsigned)n_real) continue;   // column of a neighbouring block
                            const int dx = kx - p.pad;
                            uint4 w = zero;
                            if (vec_rows) {
                                w = shifted8u(prev, cur, next, dx);
                            } else if (live) {
                                const int x0 = xb + dx;
                                uint32_t v[8];
#pragma unroll
                                for (int q = 0; q < 8; ++q) v[q] = (unsigned)(x0 + q) < (unsigned)p.W ? (uint32_t)row[x0 + q] : 0u;
                                w = make_uint4(v[0] | (v[1] << 16), v[2] | (v[3] << 16), v[4] | (v[5] << 16), v[6] | (v[7] << 16));
                            }
                            *reinterpret_cast<uint4*>(pt + n * 128 + (((uint32_t)u ^ (uint32_t)(n & 7)) << 4)) = w;
                        }
                    }
                    // the all-ones bias column and the zero rows up to the next multiple of 32
                    for (int r = n_real + gq; r < n_rows; r += GQ) {
                        const bool ones = p.has_bias && n0 + r == p.d_in;
                        const uint32_t v = ones ? 0x3F803F80u : 0u;            // bf16 1.0 twice
                        *reinterpret_cast<uint4*>(pt + r * 128 + (((uint32_t)u ^ (uint32_t)(r & 7)) << 4)) = make_uint4(v, v, v, v);
                    }
                    fence_proxy_async_smem();
                    __syncwarp();
                    if (lane == 0) mbar_arrive(&ready[s]);
                    if (t == 0) DPCLIP_TRACE_AT(1, 2 * g + 1);
                }
                if (!ok) break;
                __syncwarp();
                if (lane == 0) mbar_arrive(&xempty[b]);
            }
        }
    } else if (GRAD) {
        // ------------------------------------------------ GRAD: scale the Zb tile by the example's clip factor, in place
        const int t = threadIdx.x - 32 * (2 + EPI_WARPS + PATCH_WARPS);    // 0 .. 127
        int g = 0;
        bool ok = true;
        for (int item = blockIdx.x; item < p.n_items && ok; item += gridDim.x) {
            int e0, ne, j; decode(item, e0, ne, j);
            for (int e = e0; e < e0 + ne && ok; ++e) {
                const float f = p.clip ? __ldg(p.clip + e) : 1.f;
                // f = f_hi + f_lo (two bf16): z * f_hi + (z * f_lo) rounds the product once
                const __nv_bfloat16 fh = __float2bfloat16_rn(f);
                const __nv_bfloat16 fl = __float2bfloat16_rn(f - __bfloat162float(fh));
                const __nv_bfloat162 fh2 = __halves2bfloat162(fh, fh), fl2 = __halves2bfloat162(fl, fl);
                for (int kb = 0; kb < nkb; ++kb, ++g) {
                    const int s = g % STAGES;
                    ok = mbar_wait(&zfull[s], (g / STAGES) & 1, abort_flag, p.status);
                    if (!ok) break;
                    if (f != 1.0f) {
                        uint4* zt = reinterpret_cast<uint4*>(smem + s * STAGE_BYTES);
                        const int units = p.z_cm ? p.d_out * 8 : z_chunks * BK * 8;   // 16-byte units that hold data
                        for (int i = t; i < units; i += 32 * SCALE_WARPS) {
                            uint4 v = zt[i];
                            __nv_bfloat162* z2 = reinterpret_cast<__nv_bfloat162*>(&v);
#pragma unroll
                            for (int q = 0; q < 4; ++q) z2[q] = __hfma2(z2[q], fh2, __hmul2(z2[q], fl2));
                            zt[i] = v;
                        }
                    }
                    fence_proxy_async_smem();
                    __syncwarp();
                    if (lane == 0) mbar_arrive(&ready[s]);
                }
            }
        }
    }

    // ---------------------------------------------------- teardown
    if (*abort_flag) {
        for (int i = 0; i < 64; ++i) __nanosleep(1000);
    }
    tc_fence_before_sync();
    __syncthreads();
    if (warp == 1) { tc_fence_after_sync(); tmem_dealloc(tmem_base, 512); }
}

}  // namespace tc
}  // namespace dpclip
