// tcgen05 / TMEM / TMA kernels for bf16 layers.
//
//   gram_norm_kernel : per-example squared norms by the Gram identity
//       ||sum_t zb_t (x) a_t||_F^2 = sum_{t,s} (a_t . a_s)(zb_t . zb_s)
//     Both Gram factors of a 128 x 128 block of (t, s) pairs are accumulated in
//     tensor memory (A A^T in columns 0..127, Zb Zb^T in 128..255, fp32) from
//     K-major operand tiles fetched by TMA; the epilogue multiplies the two
//     blocks element-wise and reduces, so no Gram matrix reaches HBM.  Rows are
//     flattened (row = i*T + t), so several short examples share one block and
//     only same-example (t, s) entries are kept; blocks below the diagonal are
//     skipped and the strict upper ones counted twice.  The bias term
//     ||sum_t zb_t||^2 is the sum of the same entries of Zb Zb^T.
//
//   zta_tc_kernel : the product Zb^T diag(f) A over a range of rows, with the
//     128 x 256 fp32 output tile in tensor memory.  Both operands are read in
//     their native [row][feature] layout (MN-major UMMA operands, 128-byte
//     swizzled 64-column TMA boxes); a transform warpgroup applies the per-row
//     factor f to the Zb tile in shared memory between the TMA and the MMA.
//       GRAD mode: f = clip factor of the row's example; rows split over CTAs;
//                  the epilogue adds the tile into gW (fp32 atomics).
//       NORM mode: rows = one example, f masks rows outside it; the epilogue
//                  squares and sums the tile (Frobenius norm), so the
//                  per-example gradient never leaves the SM.
//     The bias gradient (column sums of f * Zb) is accumulated in fp32 by the
//     transform warps as they pass over the tile.
//
// Every mbarrier wait is bounded; on a timeout the CTA sets the status word in
// the workspace header and unwinds (frees its tensor memory, no trap).
#pragma once
#include "tc_common.cuh"

namespace dpclip {
namespace tc {

// ===========================================================================
// Gram kernel
// ===========================================================================
namespace gram {
constexpr int BM = 128;                       // rows per block (t and s)
constexpr int BK = 64;                        // features per stage = one 128-byte swizzle row
constexpr int STAGES = 4;
constexpr int TILE_BYTES = BM * BK * 2;       // 16 KB
constexpr int STAGE_BYTES = 2 * TILE_BYTES;   // row block + column block
constexpr int THREADS = 192;                  // warp 0 TMA, warp 1 MMA, warps 2..5 epilogue
constexpr int SMEM_BYTES = STAGES * STAGE_BYTES + 1024 /*alignment slack*/ + 256 /*barriers*/;

struct Params {
    int R, T, d_in, d_out, has_bias;
    int n_items, dense_pairs, q, ppe, kmax;
    float* sq;
    int* status;
};

// item -> (row block, column block); false when the item is empty
__device__ __forceinline__ bool decode(const Params& p, int item, int& rb, int& cb) {
    if (p.dense_pairs) {                       // T % 128 == 0: q blocks per example, q(q+1)/2 pairs
        const int e = item / p.ppe;
        int r = item % p.ppe, j = 0;
        while (r >= p.q - j) { r -= p.q - j; ++j; }
        rb = e * p.q + j;
        cb = rb + r;
        return true;
    }
    rb = item / p.kmax;
    cb = rb + item % p.kmax;
    const long last_row = min((long)rb * BM + BM - 1, (long)p.R - 1);
    const long e_last = last_row / p.T;
    const long cb_max = min((e_last + 1) * p.T - 1, (long)p.R - 1) / BM;
    return cb <= cb_max;
}
}  // namespace gram

__global__ void __launch_bounds__(gram::THREADS, 1)
gram_norm_kernel(const __grid_constant__ CUtensorMap map_a, const __grid_constant__ CUtensorMap map_z,
                 const gram::Params p) {
    using namespace gram;
    extern __shared__ uint8_t smem_raw[];
    uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
    uint64_t* full = reinterpret_cast<uint64_t*>(smem + STAGES * STAGE_BYTES);
    uint64_t* empty = full + STAGES;
    uint64_t* acc_full = empty + STAGES;
    uint64_t* acc_empty = acc_full + 2;
    uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(acc_empty + 2);
    volatile int* abort_flag = reinterpret_cast<volatile int*>(tmem_slot + 1);

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    if (threadIdx.x == 0) {
        for (int s = 0; s < STAGES; ++s) { mbar_init(&full[s], 1); mbar_init(&empty[s], 1); }
        for (int b = 0; b < 2; ++b) { mbar_init(&acc_full[b], 1); mbar_init(&acc_empty[b], 4); }
        *abort_flag = 0;
        mbar_fence_init();
        tma_prefetch_desc(&map_a);
        tma_prefetch_desc(&map_z);
    }
    if (warp == 1) { tmem_alloc(tmem_slot, 512); tmem_relinquish(); }
    tc_fence_before_sync();
    __syncthreads();
    tc_fence_after_sync();
    const uint32_t tmem_base = *tmem_slot;

    const int nk_a = (p.d_in + BK - 1) / BK, nk_z = (p.d_out + BK - 1) / BK;

    if (warp == 0) {
        // ------------------------------------------------ TMA producer
        if (lane == 0) {
            int stage = 0; uint32_t phase = 0;
            for (int item = blockIdx.x; item < p.n_items; item += gridDim.x) {
                int rb, cb;
                if (!decode(p, item, rb, cb)) continue;
                const uint32_t bytes = rb == cb ? TILE_BYTES : STAGE_BYTES;
                bool ok = true;
                for (int kb = 0; kb < nk_a + nk_z && ok; ++kb) {
                    const CUtensorMap* map = kb < nk_a ? &map_a : &map_z;
                    const int x = (kb < nk_a ? kb : kb - nk_a) * BK;
                    ok = mbar_wait(&empty[stage], phase ^ 1, abort_flag, p.status);
                    if (!ok) break;
                    uint8_t* dst = smem + stage * STAGE_BYTES;
                    mbar_arrive_expect_tx(&full[stage], bytes);
                    tma_load_2d(dst, map, &full[stage], x, rb * BM);
                    if (cb != rb) tma_load_2d(dst + TILE_BYTES, map, &full[stage], x, cb * BM);
                    if (++stage == STAGES) { stage = 0; phase ^= 1; }
                }
                if (!ok) break;
            }
        }
    } else if (warp == 1) {
        // ------------------------------------------------ MMA issuer
        if (lane == 0) {
            constexpr uint32_t idesc = make_idesc_bf16(BM, BM, 0, 0);
            int stage = 0; uint32_t phase = 0; int it = 0;
            for (int item = blockIdx.x; item < p.n_items; item += gridDim.x) {
                int rb, cb;
                if (!decode(p, item, rb, cb)) continue;
                const int buf = it & 1; const uint32_t acc_phase = (it >> 1) & 1;
                bool ok = mbar_wait(&acc_empty[buf], acc_phase ^ 1, abort_flag, p.status);
                if (!ok) break;
                tc_fence_after_sync();
                for (int kb = 0; kb < nk_a + nk_z && ok; ++kb) {
                    const bool is_a = kb < nk_a;
                    const uint32_t d_tmem = tmem_base + buf * 256 + (is_a ? 0 : 128);
                    const bool first = is_a ? kb == 0 : kb == nk_a;
                    ok = mbar_wait(&full[stage], phase, abort_flag, p.status);
                    if (!ok) break;
                    tc_fence_after_sync();
                    const uint32_t a_addr = smem_u32(smem + stage * STAGE_BYTES);
                    const uint32_t b_addr = rb == cb ? a_addr : a_addr + TILE_BYTES;
#pragma unroll
                    for (int k4 = 0; k4 < BK / 16; ++k4) {
                        // K-major, 128-byte swizzle: 8-row groups 1024 bytes apart; 16 features = 32 bytes
                        const uint64_t da = make_smem_desc_sw128(a_addr + k4 * 32, 16, 1024);
                        const uint64_t db = make_smem_desc_sw128(b_addr + k4 * 32, 16, 1024);
                        mma_bf16_ss(d_tmem, da, db, idesc, (first && k4 == 0) ? 0u : 1u);
                    }
                    mma_commit(&empty[stage]);
                    if (++stage == STAGES) { stage = 0; phase ^= 1; }
                }
                if (!ok) break;
                mma_commit(&acc_full[buf]);
                ++it;
            }
        }
    } else {
        // ------------------------------------------------ epilogue (warps 2..5)
        const int quarter = warp & 3;                       // TMEM lanes 32*quarter .. +31
        const int row_local = quarter * 32 + lane;
        int it = 0;
        for (int item = blockIdx.x; item < p.n_items; item += gridDim.x) {
            int rb, cb;
            if (!decode(p, item, rb, cb)) continue;
            const int buf = it & 1; const uint32_t acc_phase = (it >> 1) & 1;
            if (!mbar_wait(&acc_full[buf], acc_phase, abort_flag, p.status)) break;
            tc_fence_after_sync();
            const long r = (long)rb * BM + row_local;
            const bool valid = r < p.R;
            const long e = valid ? r / p.T : 0;
            // columns of this block that belong to the same example as row r
            long lo = max(e * p.T, (long)cb * BM) - (long)cb * BM;
            long hi = min(min((e + 1) * p.T, (long)p.R), (long)cb * BM + BM) - (long)cb * BM;
            if (!valid) { lo = 0; hi = 0; }
            float s = 0.f, sb = 0.f;
            const uint32_t t_row = tmem_base + ((uint32_t)(quarter * 32) << 16) + buf * 256;
#pragma unroll 1
            for (int c0 = 0; c0 < BM; c0 += 32) {
                uint32_t va[32], vz[32];
                tmem_ld_32x32(t_row + c0, va);
                tmem_ld_32x32(t_row + 128 + c0, vz);
                tmem_ld_wait();
#pragma unroll
                for (int j = 0; j < 32; ++j) {
                    const int col = c0 + j;
                    if (col >= lo && col < hi) {
                        const float z = __uint_as_float(vz[j]);
                        s = fmaf(__uint_as_float(va[j]), z, s);
                        sb += z;
                    }
                }
            }
            tc_fence_before_sync();
            __syncwarp();
            if (lane == 0) mbar_arrive(&acc_empty[buf]);
            float val = (cb > rb ? 2.f : 1.f) * (s + (p.has_bias ? sb : 0.f));
            const long e0 = __shfl_sync(0xFFFFFFFFu, e, 0);
            const bool uniform = __all_sync(0xFFFFFFFFu, valid && e == e0);
            if (uniform) {
                val = warp_sum(val);
                if (lane == 0) atomicAdd(p.sq + e0, val);
            } else if (valid && hi > lo) {
                atomicAdd(p.sq + e, val);
            }
            ++it;
        }
    }

    // ---------------------------------------------------- teardown
    if (*abort_flag) {                                      // let copies in flight land before the CTA exits
        for (int i = 0; i < 64; ++i) __nanosleep(1000);
    }
    tc_fence_before_sync();
    __syncthreads();
    if (warp == 1) { tc_fence_after_sync(); tmem_dealloc(tmem_base, 512); }
}

// ===========================================================================
// Zb^T diag(f) A kernel (GRAD and NORM modes)
// ===========================================================================
namespace zta {
constexpr int BM = 128;                        // d_out tile (UMMA M)
constexpr int BN = 256;                        // d_in tile  (UMMA N)
constexpr int BK = 64;                         // rows per stage
constexpr int STAGES = 4;
constexpr int CHUNK_BYTES = BK * 128;          // one TMA box: 64 rows x 64 bf16 columns
constexpr int A_BYTES = (BM / 64) * CHUNK_BYTES;   // Zb tile, 16 KB
constexpr int B_BYTES = (BN / 64) * CHUNK_BYTES;   // A tile, 32 KB
constexpr int STAGE_BYTES = A_BYTES + B_BYTES;     // 48 KB
constexpr int THREADS = 320;                   // warp 0 TMA, 1 MMA, 2..5 transform, 6..9 epilogue
constexpr int SMEM_BYTES = STAGES * STAGE_BYTES + 1024 + 256;

struct Params {
    int R, T, d_in, d_out;
    int norm_mode;                 // 0 = GRAD, 1 = NORM
    int tiles_m, tiles_n;
    int n_items;
    int kb_per_split;              // GRAD: 64-row blocks per item
    int do_bias;                   // GRAD: gb != NULL; NORM: has_bias
    const float* clip;             // GRAD: [B] or NULL
    float* gW; long ldg; float* gb; int use_atomic; int vec_ok;
    float* sq;                     // NORM
    int* status;
};

struct Item { int m0, n0, tn; long row_begin, row_end; int nkb; int example; };

__device__ __forceinline__ Item decode(const Params& p, int item) {
    Item w;
    const int n_tiles = p.tiles_m * p.tiles_n;
    const int tile = item % n_tiles, outer = item / n_tiles;
    w.m0 = (tile / p.tiles_n) * BM;
    w.tn = tile % p.tiles_n;
    w.n0 = w.tn * BN;
    if (p.norm_mode) {
        w.example = outer;
        w.row_begin = (long)outer * p.T;
        w.row_end = w.row_begin + p.T;
    } else {
        w.example = -1;
        w.row_begin = (long)outer * p.kb_per_split * BK;
        w.row_end = min(w.row_begin + (long)p.kb_per_split * BK, (long)p.R);
    }
    w.nkb = (int)((w.row_end - w.row_begin + BK - 1) / BK);
    return w;
}
}  // namespace zta

__global__ void __launch_bounds__(zta::THREADS, 1)
zta_tc_kernel(const __grid_constant__ CUtensorMap map_a, const __grid_constant__ CUtensorMap map_z,
              const zta::Params p) {
    using namespace zta;
    extern __shared__ uint8_t smem_raw[];
    uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
    uint64_t* full = reinterpret_cast<uint64_t*>(smem + STAGES * STAGE_BYTES);   // TMA landed
    uint64_t* ready = full + STAGES;                                             // transform done
    uint64_t* empty = ready + STAGES;                                            // MMA done with the stage
    uint64_t* acc_full = empty + STAGES;
    uint64_t* acc_empty = acc_full + 2;
    uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(acc_empty + 2);
    volatile int* abort_flag = reinterpret_cast<volatile int*>(tmem_slot + 1);

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    if (threadIdx.x == 0) {
        for (int s = 0; s < STAGES; ++s) { mbar_init(&full[s], 1); mbar_init(&ready[s], 4); mbar_init(&empty[s], 1); }
        for (int b = 0; b < 2; ++b) { mbar_init(&acc_full[b], 1); mbar_init(&acc_empty[b], 4); }
        *abort_flag = 0;
        mbar_fence_init();
        tma_prefetch_desc(&map_a);
        tma_prefetch_desc(&map_z);
    }
    if (warp == 1) { tmem_alloc(tmem_slot, 512); tmem_relinquish(); }
    tc_fence_before_sync();
    __syncthreads();
    tc_fence_after_sync();
    const uint32_t tmem_base = *tmem_slot;

    if (warp == 0) {
        // ------------------------------------------------ TMA producer
        if (lane == 0) {
            int stage = 0; uint32_t phase = 0;
            bool ok = true;
            for (int item = blockIdx.x; item < p.n_items && ok; item += gridDim.x) {
                const Item w = decode(p, item);
                for (int kb = 0; kb < w.nkb; ++kb) {
                    ok = mbar_wait(&empty[stage], phase ^ 1, abort_flag, p.status);
                    if (!ok) break;
                    uint8_t* dst = smem + stage * STAGE_BYTES;
                    const int y = (int)(w.row_begin + (long)kb * BK);
                    mbar_arrive_expect_tx(&full[stage], STAGE_BYTES);
#pragma unroll
                    for (int c = 0; c < BM / 64; ++c)
                        tma_load_2d(dst + c * CHUNK_BYTES, &map_z, &full[stage], w.m0 + c * 64, y);
#pragma unroll
                    for (int c = 0; c < BN / 64; ++c)
                        tma_load_2d(dst + A_BYTES + c * CHUNK_BYTES, &map_a, &full[stage], w.n0 + c * 64, y);
                    if (++stage == STAGES) { stage = 0; phase ^= 1; }
                }
            }
        }
    } else if (warp == 1) {
        // ------------------------------------------------ MMA issuer
        if (lane == 0) {
            constexpr uint32_t idesc = make_idesc_bf16(BM, BN, 1, 1);
            int stage = 0; uint32_t phase = 0; int it = 0;
            bool ok = true;
            for (int item = blockIdx.x; item < p.n_items && ok; item += gridDim.x) {
                const Item w = decode(p, item);
                const int buf = it & 1; const uint32_t acc_phase = (it >> 1) & 1;
                ok = mbar_wait(&acc_empty[buf], acc_phase ^ 1, abort_flag, p.status);
                if (!ok) break;
                tc_fence_after_sync();
                const uint32_t d_tmem = tmem_base + buf * BN;
                for (int kb = 0; kb < w.nkb; ++kb) {
                    ok = mbar_wait(&ready[stage], phase, abort_flag, p.status);
                    if (!ok) break;
                    tc_fence_after_sync();
                    const uint32_t a_addr = smem_u32(smem + stage * STAGE_BYTES);
                    const uint32_t b_addr = a_addr + A_BYTES;
#pragma unroll
                    for (int k4 = 0; k4 < BK / 16; ++k4) {
                        // MN-major, 128-byte swizzle: 64-column chunks CHUNK_BYTES apart (leading offset),
                        // 8-row groups 1024 bytes apart (stride offset); 16 rows = 2048 bytes
                        const uint64_t da = make_smem_desc_sw128(a_addr + k4 * 2048, CHUNK_BYTES, 1024);
                        const uint64_t db = make_smem_desc_sw128(b_addr + k4 * 2048, CHUNK_BYTES, 1024);
                        mma_bf16_ss(d_tmem, da, db, idesc, (kb == 0 && k4 == 0) ? 0u : 1u);
                    }
                    mma_commit(&empty[stage]);
                    if (++stage == STAGES) { stage = 0; phase ^= 1; }
                }
                if (!ok) break;
                mma_commit(&acc_full[buf]);
                ++it;
            }
        }
    } else if (warp < 6) {
        // ------------------------------------------------ transform (warps 2..5, 128 threads)
        // thread t owns the 8 columns [8q, 8q+8) of the Zb tile (q = t / 8) on rows (t % 8) + 8 i
        const int t = threadIdx.x - 64;
        const int q = t >> 3, rsub = t & 7;
        const int box = q >> 3, lq = q & 7;
        const uint32_t off = box * CHUNK_BYTES + rsub * 128 + ((lq ^ rsub) << 4);
        int stage = 0; uint32_t phase = 0;
        bool ok = true;
        for (int item = blockIdx.x; item < p.n_items && ok; item += gridDim.x) {
            const Item w = decode(p, item);
            const bool bias_here = p.do_bias && w.tn == 0;
            float cs[8];
#pragma unroll
            for (int j = 0; j < 8; ++j) cs[j] = 0.f;
            for (int kb = 0; kb < w.nkb; ++kb) {
                ok = mbar_wait(&full[stage], phase, abort_flag, p.status);
                if (!ok) break;
                uint8_t* zt = smem + stage * STAGE_BYTES;
                // rows of this stage: [blk0, blk0 + 64) (32-bit: B*T < 2^31 is checked on the host)
                const int blk0 = (int)w.row_begin + kb * BK;
                const int row_end = (int)w.row_end;
                const int e_first = blk0 / p.T;
                const int rem0 = blk0 - e_first * p.T;
                // fast path: the whole stage lies inside one example and inside the row range
                const bool uniform = (rem0 + BK <= p.T) && (blk0 + BK <= row_end);
                float f_uni = 1.f;
                if (uniform && p.clip) f_uni = __ldg(p.clip + e_first);
                if (!(uniform && f_uni == 1.f && !bias_here)) {
#pragma unroll
                    for (int i = 0; i < 8; ++i) {
                        float f = f_uni;
                        if (!uniform) {
                            const int rl = rsub + 8 * i;
                            if (blk0 + rl >= row_end) f = 0.f;           // rows of another example / past the end
                            else if (p.clip) f = __ldg(p.clip + e_first + (rem0 + rl) / p.T);
                        }
                        if (f != 1.f || bias_here) {
                            uint4* ptr = reinterpret_cast<uint4*>(zt + off + i * 1024);
                            uint4 v = *ptr;
                            uint32_t wds[4] = {v.x, v.y, v.z, v.w};
#pragma unroll
                            for (int h = 0; h < 4; ++h) {
                                float lo = __uint_as_float(wds[h] << 16) * f;
                                float hi = __uint_as_float(wds[h] & 0xFFFF0000u) * f;
                                cs[2 * h] += lo; cs[2 * h + 1] += hi;
                                __nv_bfloat162 pk = __floats2bfloat162_rn(lo, hi);
                                wds[h] = *reinterpret_cast<uint32_t*>(&pk);
                            }
                            if (f != 1.f) *ptr = make_uint4(wds[0], wds[1], wds[2], wds[3]);
                        }
                    }
                }
                fence_proxy_async_smem();
                __syncwarp();
                if (lane == 0) mbar_arrive(&ready[stage]);
                if (++stage == STAGES) { stage = 0; phase ^= 1; }
            }
            if (!ok) break;
            if (bias_here) {
                if (p.norm_mode) {
                    // complete the column sums over the 8 row-subsets (8 consecutive lanes), then square
                    float ssq = 0.f;
#pragma unroll
                    for (int j = 0; j < 8; ++j) {
                        float c = cs[j];
                        c += __shfl_xor_sync(0xFFFFFFFFu, c, 1);
                        c += __shfl_xor_sync(0xFFFFFFFFu, c, 2);
                        c += __shfl_xor_sync(0xFFFFFFFFu, c, 4);
                        ssq = fmaf(c, c, ssq);
                    }
                    if (rsub != 0) ssq = 0.f;
                    ssq = warp_sum(ssq);
                    if (lane == 0) atomicAdd(p.sq + w.example, ssq);
                } else {
#pragma unroll
                    for (int j = 0; j < 8; ++j) {
                        const int m = w.m0 + q * 8 + j;
                        if (m < p.d_out) atomicAdd(p.gb + m, cs[j]);
                    }
                }
            }
        }
    } else {
        // ------------------------------------------------ epilogue (warps 6..9)
        const int quarter = warp & 3;
        const int row_local = quarter * 32 + lane;
        int it = 0;
        for (int item = blockIdx.x; item < p.n_items; item += gridDim.x) {
            const Item w = decode(p, item);
            const int buf = it & 1; const uint32_t acc_phase = (it >> 1) & 1;
            if (!mbar_wait(&acc_full[buf], acc_phase, abort_flag, p.status)) break;
            tc_fence_after_sync();
            const uint32_t t_row = tmem_base + ((uint32_t)(quarter * 32) << 16) + buf * BN;
            const int m = w.m0 + row_local;
            float fro = 0.f;
#pragma unroll 1
            for (int c0 = 0; c0 < BN; c0 += 32) {
                uint32_t v[32];
                tmem_ld_32x32(t_row + c0, v);
                tmem_ld_wait();
                if (p.norm_mode) {
                    // rows/columns beyond d_out/d_in were zero-filled by TMA and add nothing
#pragma unroll
                    for (int j = 0; j < 32; ++j) { const float x = __uint_as_float(v[j]); fro = fmaf(x, x, fro); }
                } else if (m < p.d_out) {
                    const int n = w.n0 + c0;
                    float* dst = p.gW + (size_t)m * p.ldg + n;
                    if (p.vec_ok && n + 32 <= p.d_in) {
#pragma unroll
                        for (int j = 0; j < 32; j += 4) {
                            float4 x = make_float4(__uint_as_float(v[j]), __uint_as_float(v[j + 1]),
                                                   __uint_as_float(v[j + 2]), __uint_as_float(v[j + 3]));
                            if (p.use_atomic) atomicAdd(reinterpret_cast<float4*>(dst + j), x);
                            else *reinterpret_cast<float4*>(dst + j) = x;
                        }
                    } else {
#pragma unroll
                        for (int j = 0; j < 32; ++j) {
                            if (n + j < p.d_in) {
                                if (p.use_atomic) atomicAdd(dst + j, __uint_as_float(v[j]));
                                else dst[j] = __uint_as_float(v[j]);
                            }
                        }
                    }
                }
            }
            tc_fence_before_sync();
            __syncwarp();
            if (lane == 0) mbar_arrive(&acc_empty[buf]);
            if (p.norm_mode) {
                fro = warp_sum(fro);
                if (lane == 0) atomicAdd(p.sq + w.example, fro);
            }
            ++it;
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
