// Tensor-core path for fp32 layers: Zb^T diag(f) A with error-compensated tf32.
//
// fp32 inputs must come out within 1e-5, which plain tf32 (10-bit mantissa)
// cannot give.  Each operand x is split on chip into hi = x truncated to 10
// mantissa bits (what the tensor core reads of the fp32 word itself, so the
// high part needs no copy) and lo = x - hi (exact in fp32, below 2^-10 |x|,
// written to a second plane), and the product is taken as hi*hi + hi*lo + lo*hi with
// fp32 accumulation in tensor memory; the dropped lo*lo term and the tf32
// rounding of lo are both about 2^-20 relative.  Three kind::tf32 MMAs replace
// one fp32-ALU tile product at several times its speed.
//
// The tensor core adds into its fp32 accumulator with truncation, a bias
// toward zero that grows with the number of accumulation steps (about 1e-5
// relative after a few hundred).  So the accumulator is drained every FLUSH
// stages: the epilogue warps add each window into registers with ordinary
// rounded fp32 adds, and the two accumulator buffers alternate between windows.
//
// Structure as zta_tc_kernel (same Params, same GRAD / NORM modes, same
// split-row partial tiles): 128 x 128 output tile, 32-row stages; TMA brings
// the raw fp32 tiles (MN-major, 32-column boxes of 128-byte rows, 32-byte swizzle atoms), the
// transform warps apply the per-row factor to Zb in place and write its low
// plane (taking the bias column sums on the way), the epilogue warps write the
// low plane of A, one thread issues the twelve MMAs of a stage, and the
// epilogue warps drain the accumulator.
#pragma once
#include "kernels_tc.cuh"

namespace dpclip {
namespace tc {
namespace t32 {
constexpr int BM = 128, BN = 128, BK = 32;
constexpr int CHUNK_BYTES = BK * 128;                 // one TMA box: 32 rows x 32 fp32 columns
constexpr int TILE_BYTES = 4 * CHUNK_BYTES;           // 128 columns: 16 KB
constexpr int OFF_Z = 0, OFF_A = TILE_BYTES, OFF_ZLO = 2 * TILE_BYTES, OFF_ALO = 3 * TILE_BYTES;
constexpr int STAGE_BYTES = 4 * TILE_BYTES;           // raw/hi Zb, raw/hi A, lo Zb, lo A: 64 KB
constexpr int STAGES = 3, NBUF = 2;
constexpr int FLUSH = 4;                               // stages accumulated in tensor memory before a drain
constexpr int N_TRANSFORM_WARPS = 8, N_EPILOGUE_WARPS = 8;
constexpr int THREADS = 64 + 32 * (N_TRANSFORM_WARPS + N_EPILOGUE_WARPS);
constexpr int OUT_STAGE_BYTES = N_EPILOGUE_WARPS * 4096;
constexpr int SMEM_BYTES = STAGES * STAGE_BYTES + 256 + OUT_STAGE_BYTES + 1024;
constexpr uint32_t TF32_MASK = 0xFFFFE000u;           // keeps sign, exponent and 10 mantissa bits

__device__ __forceinline__ zta::Item decode(const zta::Params& p, int item) {
    zta::Item w;
    const int n_tiles = p.tiles_m * p.tiles_n;
    const int tile = item % n_tiles, outer = item / n_tiles;
    w.m0 = (tile / p.tiles_n) * BM;
    w.tn = tile % p.tiles_n;
    w.n0 = w.tn * BN;
    if (p.norm_mode) {
        w.example = outer;
        w.row_begin = outer * p.T;
        w.row_end = w.row_begin + p.T;
    } else {
        w.example = -1;
        w.row_begin = outer * p.kb_per_split * BK;
        w.row_end = min(w.row_begin + p.kb_per_split * BK, p.R);
    }
    w.nkb = (w.row_end - w.row_begin + BK - 1) / BK;
    return w;
}
}  // namespace t32

// CONV = true: the layer is a convolution given by its input feature map X [B][C][H][W] (implicit im2col).
// No TMA for the A operand: the transform warps gather element (row (i, t), column (c, ky, kx)) of the
// patch matrix from X[i][c][y' stride - pad + ky][x' stride - pad + kx] (zero outside the map) with plain
// loads, one stage ahead, and write both of its planes in the layout TMA would have produced.
struct ConvGather {
    const float* X;
    int C, H, W, kh, kw, stride, pad, Wo;
};

template <bool CONV>
__global__ void __launch_bounds__(t32::THREADS, 1)
zta_tf32_kernel(const __grid_constant__ CUtensorMap map_a, const __grid_constant__ CUtensorMap map_z,
                const zta::Params p, const ConvGather cg) {
    using namespace t32;
    using zta::Item;
    extern __shared__ uint8_t smem_raw[];
    uint8_t* smem = smem_raw + ((1024u - (smem_u32(smem_raw) & 1023u)) & 1023u);   // 1024-byte aligned; an offset from the array keeps the accesses in the shared state space
    uint64_t* full = reinterpret_cast<uint64_t*>(smem + STAGES * STAGE_BYTES);   // TMA landed
    uint64_t* ready = full + STAGES;                                             // hi/lo planes written
    uint64_t* empty = ready + STAGES;                                            // MMA done with the stage
    uint64_t* acc_full = empty + STAGES;
    uint64_t* acc_empty = acc_full + 2;
    uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(acc_empty + 2);
    volatile int* abort_flag = reinterpret_cast<volatile int*>(tmem_slot + 1);
    float4* out_stage = reinterpret_cast<float4*>(smem + STAGES * STAGE_BYTES + 256);

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    if (threadIdx.x == 0) {
        for (int s = 0; s < STAGES; ++s) {
            mbar_init(&full[s], 1); mbar_init(&ready[s], CONV ? N_TRANSFORM_WARPS : N_TRANSFORM_WARPS + N_EPILOGUE_WARPS);
            mbar_init(&empty[s], 1);
        }
        for (int b = 0; b < 2; ++b) { mbar_init(&acc_full[b], 1); mbar_init(&acc_empty[b], N_EPILOGUE_WARPS); }
        *abort_flag = 0;
        mbar_fence_init();
        tma_prefetch_desc(&map_a);
        tma_prefetch_desc(&map_z);
    }
    if (warp == 1) { tmem_alloc(tmem_slot, 256); tmem_relinquish(); }
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
                    const int y = w.row_begin + kb * BK;
                    mbar_arrive_expect_tx(&full[stage], CONV ? TILE_BYTES : 2 * TILE_BYTES);
#pragma unroll
                    for (int c = 0; c < 4; ++c)
                        tma_load_2d(dst + OFF_Z + c * CHUNK_BYTES, &map_z, &full[stage], w.m0 + c * 32, y);
                    if (!CONV) {
#pragma unroll
                        for (int c = 0; c < 4; ++c)
                            tma_load_2d(dst + OFF_A + c * CHUNK_BYTES, &map_a, &full[stage], w.n0 + c * 32, y);
                    }
                    if (++stage == STAGES) { stage = 0; phase ^= 1; }
                }
            }
        }
    } else if (warp == 1) {
        // ------------------------------------------------ MMA issuer
        if (lane == 0) {
            constexpr uint32_t idesc = make_idesc_tf32(BM, BN, 1, 1);
            int stage = 0; uint32_t phase = 0; int it = 0;
            bool ok = true;
            for (int item = blockIdx.x; item < p.n_items && ok; item += gridDim.x) {
                const Item w = decode(p, item);
                uint32_t d_tmem = tmem_base;
                int buf = 0;
                for (int kb = 0; kb < w.nkb; ++kb) {
                    const bool window_start = (kb % FLUSH) == 0;
                    if (window_start) {
                        // a fresh accumulator every FLUSH stages: the epilogue warps add the windows up
                        buf = it % NBUF;
                        ok = mbar_wait(&acc_empty[buf], ((it / NBUF) & 1) ^ 1, abort_flag, p.status);
                        if (!ok) break;
                        tc_fence_after_sync();
                        d_tmem = tmem_base + buf * BN;
                    }
                    ok = mbar_wait(&ready[stage], phase, abort_flag, p.status);
                    if (!ok) break;
                    tc_fence_after_sync();
                    const uint32_t base = smem_u32(smem + stage * STAGE_BYTES);
#pragma unroll
                    for (int k8 = 0; k8 < BK / 8; ++k8) {
                        // MN-major fp32 operands, 128-byte swizzle on 32-byte atoms: 32-column chunks
                        // CHUNK_BYTES apart, 4-row groups 512 bytes apart, 8 rows per K = 8 instruction
                        const uint64_t zh = make_smem_desc_sw128_atom32(base + OFF_Z + k8 * 1024, CHUNK_BYTES, 512);
                        const uint64_t zl = make_smem_desc_sw128_atom32(base + OFF_ZLO + k8 * 1024, CHUNK_BYTES, 512);
                        const uint64_t ah = make_smem_desc_sw128_atom32(base + OFF_A + k8 * 1024, CHUNK_BYTES, 512);
                        const uint64_t al = make_smem_desc_sw128_atom32(base + OFF_ALO + k8 * 1024, CHUNK_BYTES, 512);
                        mma_tf32_ss(d_tmem, zl, ah, idesc, (window_start && k8 == 0) ? 0u : 1u);   // small terms first
                        mma_tf32_ss(d_tmem, zh, al, idesc, 1u);
                        mma_tf32_ss(d_tmem, zh, ah, idesc, 1u);
                    }
                    mma_commit(&empty[stage]);
                    if (++stage == STAGES) { stage = 0; phase ^= 1; }
                    if ((kb % FLUSH) == FLUSH - 1 || kb == w.nkb - 1) { mma_commit(&acc_full[buf]); ++it; }
                }
            }
        }
    } else if (warp < 2 + N_TRANSFORM_WARPS) {
#include "kernels_tf32_transform.inc"
    } else {
#include "kernels_tf32_epilogue.inc"
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
