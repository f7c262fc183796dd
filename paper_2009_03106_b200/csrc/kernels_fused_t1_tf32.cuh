// Tensor-core second launch of the fused T = 1 step for fp32 models.
//
// Same contract as t1_all_grads_kernel (factors rebuilt per CTA from the layer
// norms, clipped sums of ALL layers, Philox noise added before the single
// store of each output), but the products run as error-compensated tf32 on
// tcgen05: per layer, 128 x 128 output tiles with K = B rows, operands brought
// by TMA as 32-row stages and split on chip into a tf32 high part and an fp32
// low part (the transform warps take the zb tile: diag(c), low plane, bias
// column sums; the epilogue warps take the A tile), three MMAs per K = 8 step.
//
// The tensor core reads an fp32 word as tf32 by ignoring its low 13 mantissa
// bits, so the high part needs no copy of its own: the (scaled) operand stays
// where it is and only low = x - truncate(x) is written to a second plane.
//
// The epilogue warps draw the noise of their outputs while the MMAs run and
// start their register accumulators from it; when the tile is done they add
// the accumulator and store through a shared-memory transpose.
//
// A layer with at most 16 outputs ("thin", e.g. a classifier head) need not
// have zb rows that TMA can address: the transform warps fetch its few zb
// values with plain loads and build the operand planes themselves; everything
// else is the same tile pipeline.
#pragma once
#include "kernels_fused_t1.cuh"
#include "kernels_tf32.cuh"

namespace dpclip {
namespace tc {
namespace f1 {
using t32::BK;
using t32::BM;
using t32::BN;
using t32::CHUNK_BYTES;
using t32::FLUSH;
using t32::NBUF;
using t32::OFF_A;
using t32::OFF_ALO;
using t32::OFF_Z;
using t32::OFF_ZLO;
using t32::STAGE_BYTES;
using t32::STAGES;
using t32::TF32_MASK;
using t32::TILE_BYTES;
constexpr int N_TRANSFORM_WARPS = 8, N_EPILOGUE_WARPS = 8;
constexpr int THREADS = 64 + 32 * (N_TRANSFORM_WARPS + N_EPILOGUE_WARPS);
constexpr int OUT_STAGE_BYTES = N_EPILOGUE_WARPS * 2048;        // 32 rows x 16 columns per warp
constexpr int CLIP_BYTES = FUSED_MAX_B * 4;
constexpr int SMEM_BYTES = STAGES * STAGE_BYTES + 256 + OUT_STAGE_BYTES + CLIP_BYTES + 1024;
constexpr int THIN_MAX_OUT = 16;

struct Params {
    FusedT1Params base;
    CUtensorMap map_a[FUSED_MAX_LAYERS];
    CUtensorMap map_z[FUSED_MAX_LAYERS];
    int thin[FUSED_MAX_LAYERS];          // 1: zb fetched by plain loads (d_out <= 16), no tensor map for it
    int item_begin[FUSED_MAX_LAYERS];
    int tiles_n[FUSED_MAX_LAYERS];
    int total_items;
    int* status;
    unsigned int* grid_counter;          // one-launch form: arrivals at the grid-wide barrier (self-resetting)
};

struct Item { int l, thin, m0, n0, tn; };

__device__ __forceinline__ Item decode(const Params& q, int item) {
    Item w;
    int l = 0;
    while (l + 1 < q.base.L && item >= q.item_begin[l + 1]) ++l;
    const int local = item - q.item_begin[l];
    w.l = l; w.thin = q.thin[l];
    w.m0 = (local / q.tiles_n[l]) * BM; w.tn = local % q.tiles_n[l]; w.n0 = w.tn * BN;
    return w;
}

// standard normal number e of noise stream sid
__device__ __forceinline__ float philox_normal(size_t e, unsigned long long sid, uint32_t k0, uint32_t k1) {
    const size_t q = e >> 2;
    PhiloxBlock b = philox_block((uint32_t)q, (uint32_t)(q >> 32), (uint32_t)sid, (uint32_t)(sid >> 32), k0, k1);
    float za, zb;
    box_muller(b.v[e & 2], b.v[(e & 2) + 1], za, zb);
    return (e & 1) ? zb : za;
}
// Sums of squares of two rows (one of A, one of Zb), taken by one warp.  All loads of a pass (up to
// eight 128-bit loads per lane and row) are issued before the first value is used: the rows are short and
// the time is load latency.  Partial sums are returned per lane (warp_sum them).
// Four consecutive elements as loaded (conversion is left to the consumer, so that a batch of predicated
// loads stays a batch of plain load instructions).
__device__ __forceinline__ float4 load_raw4(const float* p) { return *reinterpret_cast<const float4*>(p); }
__device__ __forceinline__ uint2 load_raw4(const __nv_bfloat16* p) { return *reinterpret_cast<const uint2*>(p); }
__device__ __forceinline__ float sumsq_raw4(float4 v) { return (v.x * v.x + v.y * v.y) + (v.z * v.z + v.w * v.w); }
__device__ __forceinline__ float sumsq_raw4(uint2 r) {
    const float x = __uint_as_float(r.x << 16), y = __uint_as_float(r.x & 0xFFFF0000u);
    const float z = __uint_as_float(r.y << 16), w = __uint_as_float(r.y & 0xFFFF0000u);
    return (x * x + y * y) + (z * z + w * w);
}
template <typename T> struct Raw4 { using type = float4; };
template <> struct Raw4<__nv_bfloat16> { using type = uint2; };

template <typename T>
__device__ __forceinline__ void warp_rows_sumsq(const T* __restrict__ ra, int na, bool vec_a,
                                                const T* __restrict__ rz, int nz, bool vec_z, int lane,
                                                float& sa, float& sz) {
    using R = typename Raw4<T>::type;
    sa = 0.f; sz = 0.f;
    const int nva = vec_a ? na >> 2 : 0, nvz = vec_z ? nz >> 2 : 0;
    const int passes = (max(nva, nvz) + 255) >> 8;
    for (int ps = 0; ps < passes; ++ps) {
        R va[8], vz[8];
#pragma unroll
        for (int u = 0; u < 8; ++u) {
            const int j = (ps << 8) + (u << 5) + lane;
            va[u] = R{}; vz[u] = R{};
            if (j < nva) va[u] = load_raw4(ra + 4 * j);
            if (j < nvz) vz[u] = load_raw4(rz + 4 * j);
        }
#pragma unroll
        for (int u = 0; u < 8; ++u) { sa += sumsq_raw4(va[u]); sz += sumsq_raw4(vz[u]); }
    }
    // tails, and rows that cannot take vector loads
    for (int j0 = nva << 2; j0 < na; j0 += 128) {
        float v[4];
#pragma unroll
        for (int u = 0; u < 4; ++u) { const int j = j0 + (u << 5) + lane; v[u] = j < na ? to_f32(ra[j]) : 0.f; }
        sa += (v[0] * v[0] + v[1] * v[1]) + (v[2] * v[2] + v[3] * v[3]);
    }
    for (int j0 = nvz << 2; j0 < nz; j0 += 128) {
        float v[4];
#pragma unroll
        for (int u = 0; u < 4; ++u) { const int j = j0 + (u << 5) + lane; v[u] = j < nz ? to_f32(rz[j]) : 0.f; }
        sz += (v[0] * v[0] + v[1] * v[1]) + (v[2] * v[2] + v[3] * v[3]);
    }
}

__device__ __forceinline__ void named_barrier_sync(int id, int threads) {
    asm volatile("bar.sync %0, %1;" ::"r"(id), "r"(threads) : "memory");
}

// Grid-wide barrier of a cooperative launch (all CTAs resident).  Every CTA adds one to the counter on
// arrival and one more when it leaves the kernel; the counter wraps to zero at 2 * gridDim.x, so each
// launch finds it at zero.  The wait is bounded like every other wait here.
__device__ __forceinline__ bool grid_barrier_arrive_and_wait(unsigned int* ctr, volatile int* abort_flag,
                                                             int* status_word) {
    __threadfence();
    atomicInc(ctr, 2u * gridDim.x - 1u);
    const uint64_t t0 = global_ns();
    uint32_t spins = 0;
    while (true) {
        uint32_t v;
        asm volatile("ld.acquire.gpu.global.u32 %0, [%1];" : "=r"(v) : "l"(ctr) : "memory");
        if (v >= gridDim.x) return true;
        if ((++spins & 0x3F) == 0) {
            if (*abort_flag) return false;
            if (global_ns() - t0 > kWaitLimitNs) {
                *abort_flag = 1;
                if (status_word) atomicExch(status_word, (int)DPCLIP_ERR_TIMEOUT);
                return false;
            }
        }
    }
}
}  // namespace f1

// ONE_LAUNCH = false: second launch of the step (layer norms already in p.sq).
// ONE_LAUNCH = true : the whole step in one cooperative launch.  TMA and the noise generator start at
//                     once (neither depends on the factors); meanwhile the transform warps take the layer
//                     norms of the rows dealt to this CTA, meet the other CTAs at a grid-wide barrier,
//                     rebuild the factors and only then start on the staged tiles.
// T = float: error-compensated tf32 as described above.  T = __nv_bfloat16: the same pipeline with one
// kind::f16 MMA per K = 16 step and no low planes (products of bf16 inputs are exact in fp32; the only
// rounding is that of c * zb back to bf16); a stage holds 32 rows as two 64-column boxes per operand.
template <bool ONE_LAUNCH, typename T = float>
__global__ void __launch_bounds__(f1::THREADS, 1)
t1_all_grads_tf32_kernel(const __grid_constant__ f1::Params q) {
    using namespace f1;
    constexpr bool BF16 = sizeof(T) == 2;
    constexpr int BOXES = BF16 ? 2 : 4, BOX_COLS = BF16 ? 64 : 32;          // TMA boxes per 128-column tile
    const FusedT1Params& p = q.base;
    extern __shared__ uint8_t smem_raw[];
    uint8_t* smem = smem_raw + ((1024u - (smem_u32(smem_raw) & 1023u)) & 1023u);   // 1024-byte aligned; an offset from the array keeps the accesses in the shared state space
    uint64_t* full = reinterpret_cast<uint64_t*>(smem + STAGES * STAGE_BYTES);   // TMA landed
    uint64_t* ready = full + STAGES;                                             // low planes written (all 16 warps)
    uint64_t* empty = ready + STAGES;                                            // MMA done with the stage
    uint64_t* acc_full = empty + STAGES;
    uint64_t* acc_empty = acc_full + 2;
    uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(acc_empty + 2);
    volatile int* abort_flag = reinterpret_cast<volatile int*>(tmem_slot + 1);
    float4* out_stage = reinterpret_cast<float4*>(smem + STAGES * STAGE_BYTES + 256);
    float* clip_s = reinterpret_cast<float*>(smem + STAGES * STAGE_BYTES + 256 + OUT_STAGE_BYTES);

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    if (threadIdx.x == 0) {
        DPCLIP_TRACE_AT(0, 255);
        for (int s = 0; s < STAGES; ++s) {
            mbar_init(&full[s], 1); mbar_init(&ready[s], BF16 ? N_TRANSFORM_WARPS : N_TRANSFORM_WARPS + N_EPILOGUE_WARPS);
            mbar_init(&empty[s], 1);
        }
        for (int b = 0; b < 2; ++b) { mbar_init(&acc_full[b], 1); mbar_init(&acc_empty[b], N_EPILOGUE_WARPS); }
        *abort_flag = 0;
        mbar_fence_init();
    }
    if (warp == 0 && lane < p.L) {
        tma_prefetch_desc(&q.map_a[lane]);
        if (!q.thin[lane]) tma_prefetch_desc(&q.map_z[lane]);
    }
    if (warp == 1) { tmem_alloc(tmem_slot, 256); tmem_relinquish(); }
    // factors, rebuilt by every CTA from the layer norms (L * B floats, L2-resident)
    if (!ONE_LAUNCH)
    for (int i = threadIdx.x; i < p.B; i += THREADS) {
        if (p.clip_in) { clip_s[i] = p.clip_in[i]; continue; }
        float s = 0.f;
        for (int l = 0; l < p.L; ++l) s += p.sq[(size_t)l * p.B + i];
        const float n = sqrtf(s);
        const float c = n > p.C ? p.C / n : 1.0f;
        clip_s[i] = c;
        if (blockIdx.x == 0) { p.clip[i] = c; if (p.norms) p.norms[i] = n; }
    }
    tc_fence_before_sync();
    __syncthreads();
    tc_fence_after_sync();
    const uint32_t tmem_base = *tmem_slot;
    const int nkb = (p.B + BK - 1) / BK;

    if (warp == 0) {
        // ------------------------------------------------ TMA producer
        // one-launch form: the tiles are not needed before the factors exist, so the tile loads start when
        // the norm phase has its rows (its few loads then do not queue behind megabytes of tile traffic,
        // and the tile loads hit L2)
        if (ONE_LAUNCH) named_barrier_sync(2, 32 + 32 * N_TRANSFORM_WARPS);
        if (lane == 0) {
            int stage = 0; uint32_t phase = 0;
            bool ok = true;
            [[maybe_unused]] int tr = 0;
            DPCLIP_TRACE_AT(0, 254);
            for (int item = blockIdx.x; item < q.total_items && ok; item += gridDim.x) {
                const Item w = decode(q, item);
                const CUtensorMap* ma = &q.map_a[w.l];
                const CUtensorMap* mz = &q.map_z[w.l];
                for (int kb = 0; kb < nkb; ++kb) {
                    ok = mbar_wait(&empty[stage], phase ^ 1, abort_flag, q.status);
                    if (!ok) break;
                    uint8_t* dst = smem + stage * STAGE_BYTES;
                    DPCLIP_TRACE_AT(0, tr); ++tr;
                    mbar_arrive_expect_tx(&full[stage], (w.thin ? 1 : 2) * BOXES * CHUNK_BYTES);
                    if (!w.thin) {
#pragma unroll
                        for (int c = 0; c < BOXES; ++c)
                            tma_load_2d(dst + OFF_Z + c * CHUNK_BYTES, mz, &full[stage], w.m0 + c * BOX_COLS, kb * BK);
                    }
#pragma unroll
                    for (int c = 0; c < BOXES; ++c)
                        tma_load_2d(dst + OFF_A + c * CHUNK_BYTES, ma, &full[stage], w.n0 + c * BOX_COLS, kb * BK);
                    if (++stage == STAGES) { stage = 0; phase ^= 1; }
                }
            }
        }
    } else if (warp == 1) {
        // ------------------------------------------------ MMA issuer
        if (lane == 0) {
            constexpr uint32_t idesc = BF16 ? make_idesc_bf16(BM, BN, 1, 1) : make_idesc_tf32(BM, BN, 1, 1);
            int stage = 0; uint32_t phase = 0; int it = 0;
            bool ok = true;
            [[maybe_unused]] int tr = 0;
            for (int item = blockIdx.x; item < q.total_items && ok; item += gridDim.x) {
                const Item w = decode(q, item);
                uint32_t d_tmem = tmem_base;
                int buf = 0;
                for (int kb = 0; kb < nkb; ++kb) {
                    const bool window_start = (kb % FLUSH) == 0;
                    if (window_start) {
                        buf = it % NBUF;
                        ok = mbar_wait(&acc_empty[buf], ((it / NBUF) & 1) ^ 1, abort_flag, q.status);
                        if (!ok) break;
                        tc_fence_after_sync();
                        d_tmem = tmem_base + buf * BN;
                    }
                    ok = mbar_wait(&ready[stage], phase, abort_flag, q.status);
                    if (!ok) break;
                    tc_fence_after_sync();
                    DPCLIP_TRACE_AT(2, tr); ++tr;
                    const uint32_t base = smem_u32(smem + stage * STAGE_BYTES);
                    if (BF16) {
#pragma unroll
                        for (int k16 = 0; k16 < BK / 16; ++k16) {
                            // MN-major bf16, 128-byte swizzle: 64-column chunks CHUNK_BYTES apart, 8-row groups
                            // 1024 bytes apart, 16 rows per K = 16 instruction
                            const uint64_t dz = make_smem_desc_sw128(base + OFF_Z + k16 * 2048, CHUNK_BYTES, 1024);
                            const uint64_t da = make_smem_desc_sw128(base + OFF_A + k16 * 2048, CHUNK_BYTES, 1024);
                            mma_bf16_ss(d_tmem, dz, da, idesc, (window_start && k16 == 0) ? 0u : 1u);
                        }
                    } else
#pragma unroll
                    for (int k8 = 0; k8 < BK / 8; ++k8) {
                        // the raw planes double as the high parts (the low 13 bits are not read)
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
                    if ((kb % FLUSH) == FLUSH - 1 || kb == nkb - 1) { mma_commit(&acc_full[buf]); ++it; }
                }
            }
        }
    } else if (warp < 2 + N_TRANSFORM_WARPS) {
        if constexpr (BF16) {
#include "kernels_fused_t1_bf16_transform.inc"
        } else {
#include "kernels_fused_t1_tf32_transform.inc"
        }
    } else {
#include "kernels_fused_t1_tf32_epilogue.inc"
    }

    // ---------------------------------------------------- teardown
    if (*abort_flag) {
        for (int i = 0; i < 64; ++i) __nanosleep(1000);
    }
    tc_fence_before_sync();
    __syncthreads();
    if (warp == 1) { tc_fence_after_sync(); tmem_dealloc(tmem_base, 256); }
    if (ONE_LAUNCH && threadIdx.x == 0) atomicInc(q.grid_counter, 2u * gridDim.x - 1u);   // leave: see the barrier
}

}  // namespace tc
}  // namespace dpclip
