// Clipped sums Zb^T diag(c) A (Algorithm 1, the reweighted backward pass) of up to eight layers in ONE
// launch, on CTA PAIRS (tcgen05.mma.cta_group::2), with the work cut stream-K fashion: bf16, sm_100a.
//
// Why pairs.  The single-CTA kernel (zta_tc_kernel) is bound by its shared-memory port: per 16 rows of a
// 256 x 256 tile, TMA writes 16 KB of operands, the transform warps read and rewrite 8 KB of Zb to apply
// diag(c), and the two 128 x 256 x 16 MMAs read 24 KB: 56 KB for 256 tensor clocks at 128 B/clk.  A pair of
// CTAs on the two SMs of a TPC works on ONE 512 (d_out) x 256 (d_in) tile: each CTA holds 256 Zb columns
// (two 128-row M sub-tiles) and only HALF of the A columns (128); an MMA of the pair (M = 256, N = 256) takes
// each CTA's own M sub-tile and the two N halves, one from each shared memory.  And the per-row factor is
// applied to the A half (128 columns) instead of the Zb tile (256 columns): Zb^T diag(c) A = Zb^T (diag(c) A).
// Per 16 rows and CTA: TMA writes 8 + 4 KB, the transform rewrites 4 KB (8 KB of traffic), the two MMAs read
// 2 x (4 + 4) KB.
//
// How the work is cut.  All layers of the launch have the same rows (B*T), so a tile of any layer is the same
// amount of work: S = ceil(B*T / 64) stages.  Tiles that read the same operand columns must stream the same
// rows AT THE SAME TIME, or every one of them fetches those rows from HBM again (tile-major stream-K over the
// seven sequence-model layers: 319 us, twice the DRAM traffic).  So tiles are packed into "super-layers" of W
// tiles (a sub-grid of one layer, or several narrow layers side by side), pairs into gangs of W (pair j of a
// gang takes tile j of the super-layer the gang is on, all W in step on the same rows), and the sequence of
// (super-layer, stage) units is cut into equal runs, one per gang: every gang is busy for the same time
// whatever the number of tiles (B*T = 32768, seven layers = 32 tiles = 4 super-layers of 8: nine gangs x 228
// stages, where one launch per layer with nine row slices pays set-up, pipeline fill and the accumulator
// drain four times).  A run crosses at most ceil(U / S) super-layer boundaries; at each one the pair drains
// its accumulator into a partial tile ("segment") and starts its tile of the next super-layer.
// reduce_segments_kernel then adds the segments of every tile in a fixed order (bit-reproducible), adds the
// noise and writes gW / gb.  Segment s(u) of unit u = u / S + u / U - u / lcm(S, U): the number of
// super-layer and run boundaries in (0, u]; pair j's partial tile is slot s(u) * W + j.  W = 1 is plain
// tile-major stream-K (used when the tile counts fit no common gang width).
//
// Roles per CTA (same warp layout in both CTAs): warp 0 = TMA producer of this CTA's operands (plain
// per-CTA tile loads into its own shared memory, completion on its own barrier: nothing is multicast);
// warp 1 = MMA issuer -- rank 0 only, rank 1's warp 1 just owns its half of the tensor-memory allocation;
// 8 transform warps: scale this CTA's A half by the row's factor (bf16, one rounding), then arrive on rank
// 0's `ready` barrier (a remote arrive for rank 1); 8 epilogue warps: during the main loop (when a layer of
// the launch has a bias) the column sums sum_rows c * zb straight from the untouched Zb tile, in fp32, for the
// stages dealt to this n-tile -- beside the transform warps and the MMAs: they only hold up the REFILL of the
// stage (`zfree`, local) -- and at the end of a segment the drain of this CTA's accumulator (256 d_out rows x
// 256 d_in columns fp32 = all 512 tensor-memory columns).
// Barriers: full[s] (local, TMA bytes) -> ready[s] (in rank 0, 16 warp arrivals from both CTAs) -> MMAs
// -> empty[s] / acc_full (tcgen05.commit with an arrival in BOTH CTAs) -> acc_empty (in rank 0, 16 arrivals);
// the producer refills stage s after empty[s] and zfree[s].
// Every wait is bounded; a CTA that gives up sets the status word, unwinds, and still takes part in the
// closing cluster barrier, so its partner neither waits for ever nor touches shared memory of a CTA that
// has exited.
//
// What the timeline showed on the way: a remote mbarrier arrive spelled .release.cluster holds its thread for
// 0.7-1.6 us (the default form does not); with the MMAs taken out the pipeline streams a 48 KB stage every
// 0.7 us per SM, with them a stage takes 0.9 us although its eight MMAs need 0.65 us -- operand reads and TMA
// writes meet at the shared-memory port -- and with 18 instead of 74 pairs active 0.67 us; L2 prefetches 2-8
// stages beyond the ring made it slower (they are requests too); the bias sums on the transform warps cost
// 10 us per layer, on the otherwise idle epilogue warps 4.
#pragma once
#include "kernels_tc.cuh"

namespace dpclip {
namespace tc {
namespace ztp {
constexpr int BM_CTA = 256;                    // d_out columns of Zb per CTA (two M sub-tiles of 128)
constexpr int BM = 2 * BM_CTA;                 // d_out extent of a pair tile
constexpr int BN = 256;                        // d_in extent of a pair tile (UMMA N)
constexpr int BN_CTA = BN / 2;                 // A columns per CTA
constexpr int BK = 64;                         // rows per stage
constexpr int CHUNK_BYTES = BK * 128;          // one TMA box: BK rows x 64 bf16 columns
constexpr int Z_BYTES = (BM_CTA / 64) * CHUNK_BYTES;     // 32 KB
constexpr int A_BYTES = (BN_CTA / 64) * CHUNK_BYTES;     // 16 KB
constexpr int STAGE_BYTES = Z_BYTES + A_BYTES;           // 48 KB
constexpr int STAGES = 4;
constexpr int N_TRANSFORM_WARPS = 8, N_EPILOGUE_WARPS = 8;
constexpr int THREADS = 64 + 32 * (N_TRANSFORM_WARPS + N_EPILOGUE_WARPS);
constexpr int OUT_STAGE_BYTES = N_EPILOGUE_WARPS * 4096;
constexpr int SMEM_BYTES = STAGES * STAGE_BYTES + 256 + OUT_STAGE_BYTES + 1024;
constexpr int MAX_LAYERS = zta::MAX_LAYERS;
constexpr size_t SEG_ELEMS = (size_t)BM * BN;  // fp32 elements of a segment's partial tile

struct Layer {
    int d_in, d_out;
    int tiles_n;                   // pair tiles along d_in
    int tile_base, tiles;          // this layer's tiles are tile_base .. tile_base + tiles - 1 of the launch
    int do_bias;
    const float* clip;             // [B] factors of THIS layer, or NULL (all ones): one vector for the whole model under
                                   // global clipping, one per layer under per-layer clipping
    float* gW; float* gb;          // outputs (dense rows: ldg = d_in for the noise; see ldg)
    long ldg; int vec_ok;
    uint32_t sw0, sw1, sb0, sb1;   // noise streams of gW and gb
};

constexpr int MAX_TILES = 256;                 // tiles of all layers of a launch (table size)

struct Params {
    int R, T;                      // rows B*T of every layer, rows per example
    int S;                         // stages per tile = ceil(R / BK)
    int n_layers, G;               // tiles of all layers
    int W, n_super;                // gang width; super-layers of up to W tiles
    int U;                         // units (super-layer stages) per gang
    long total, lcm;               // n_super * S; lcm(S, U)
    short super_tile[MAX_TILES];   // [n_super][W]: tile of the launch at position j of super-layer s, or -1
    short tile_slot[MAX_TILES];    // [G]: s * W + j of every tile
    int seg_first[MAX_TILES];      // [G]: slot of the tile's first segment (first segment of its super-layer * W + j)
    short seg_count[MAX_TILES];    // [G]: segments its stages are cut into; they lie W slots apart
    unsigned char tile_layer[MAX_TILES];   // [G]: layer of the launch a tile belongs to
    int any_bias;
    long n_segments;               // partial tiles the workspace holds (range checks of the debug build)
    float* part;                   // [n_segments][BM][BN] fp32
    float* bias_part;              // [n_segments][BM] fp32, or NULL when no layer has a bias
    int* status;
    float noise_scale; uint32_t k0, k1;
    Layer layer[MAX_LAYERS];
};

__device__ __forceinline__ float row_factor(const Params& p, const float* clip, int e) {
    if (!DPCLIP_IN_RANGE(e, (p.R + p.T - 1) / p.T, p.status)) return 0.f;
    return clip ? __ldg(clip + e) : 1.f;
}

__host__ __device__ __forceinline__ long segment_of(long u, int S, int U, long lcm) { return u / S + u / U - u / lcm; }

struct Seg { int layer, m0, n0, tn, kb0, kb1; long slot; };       // layer < 0: this pair has no tile in the segment

// the segment that starts at unit u of a run that ends before unit u_end, for pair j of the gang
__device__ __forceinline__ Seg segment_at(const Params& p, long u, long u_end, int j) {
    Seg s;
    const int sl = (int)(u / p.S);
    s.kb0 = (int)(u - (long)sl * p.S);
    const long left = u_end - u;
    s.kb1 = (int)min((long)p.S, s.kb0 + left);
    const int g = p.super_tile[sl * p.W + j];
    s.layer = -1; s.m0 = s.n0 = s.tn = 0; s.slot = 0;
    if (g < 0) return s;
    int l = 0;
#pragma unroll 1
    while (l + 1 < p.n_layers && g >= p.layer[l + 1].tile_base) ++l;
    s.layer = l;
    const int tile = g - p.layer[l].tile_base;
    const int tm = tile / p.layer[l].tiles_n;
    s.tn = tile - tm * p.layer[l].tiles_n;
    s.m0 = tm * BM;
    s.n0 = s.tn * BN;
    s.slot = segment_of(u, p.S, p.U, p.lcm) * p.W + j;
    return s;
}
}  // namespace ztp

__global__ void __cluster_dims__(2, 1, 1) __launch_bounds__(ztp::THREADS, 1)
zta_pair_kernel(const __grid_constant__ zta::Maps maps, const __grid_constant__ ztp::Params p) {
    using namespace ztp;
    extern __shared__ uint8_t smem_raw[];
    // 1024-byte aligned by an OFFSET from the array (keeps the accesses in the shared state space); the offset
    // is the same in both CTAs (same kernel, same static layout), which the pair's descriptors rely on
    uint8_t* smem = smem_raw + ((1024u - (smem_u32(smem_raw) & 1023u)) & 1023u);
    uint64_t* full = reinterpret_cast<uint64_t*>(smem + STAGES * STAGE_BYTES);   // TMA landed (this CTA)
    uint64_t* ready = full + STAGES;                                             // transform done (rank 0's is used)
    uint64_t* empty = ready + STAGES;                                            // MMAs done with the stage (each CTA's own)
    uint64_t* acc_full = empty + STAGES;                                         // accumulator complete (each CTA's own)
    uint64_t* acc_empty = acc_full + 1;                                          // accumulator drained (rank 0's is used)
    uint64_t* zfree = acc_empty + 1;                                             // bias warps done reading the Zb tile (own)
    uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(zfree + STAGES);
    volatile int* abort_flag = reinterpret_cast<volatile int*>(tmem_slot + 1);
    float4* out_stage = reinterpret_cast<float4*>(smem + STAGES * STAGE_BYTES + 256);

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const uint32_t rank = cluster_ctarank();                  // 0 = issues the MMAs
    const int pair = blockIdx.x >> 1;
    const int gang = pair / p.W, gj = pair - gang * p.W;      // pair gj of its gang
    const long u_begin = min((long)gang * p.U, p.total), u_end = min(u_begin + p.U, p.total);   // the gang's run
    if (threadIdx.x == 0) {
        for (int s = 0; s < STAGES; ++s) {
            mbar_init(&full[s], 1);
            mbar_init(&ready[s], 2 * N_TRANSFORM_WARPS);
            mbar_init(&empty[s], 1);
            // with a bias the epilogue warps read every stage's Zb tile (column sums): they hold up the refill of
            // the stage, not the MMAs
            mbar_init(&zfree[s], N_EPILOGUE_WARPS);
        }
        mbar_init(acc_full, 1); mbar_init(acc_empty, 2 * N_EPILOGUE_WARPS);
        *abort_flag = 0;
        mbar_fence_init();
        for (int l = 0; l < p.n_layers; ++l) { tma_prefetch_desc(&maps.a[l]); tma_prefetch_desc(&maps.z[l]); }
    }
    if (warp == 1) { tmem_alloc_pair(tmem_slot, 512); tmem_relinquish_pair(); }
    tc_fence_before_sync();
    cluster_sync_all();             // both CTAs' barriers initialised and tensor memory allocated before anyone proceeds
    tc_fence_after_sync();
    const uint32_t tmem_base = *tmem_slot;
    // When the launch overlaps the tail of the kernel that computes the factors, only the loads of the layers'
    // inputs (which no kernel of a step writes) may run ahead: the warps that read the factors or write the
    // workspace wait for that kernel here.
    if (warp >= 2) griddep_wait();

    if (warp == 0) {
        // ------------------------------------------------ TMA producer (each CTA loads its own operands)
        if (lane == 0) {
            int stage = 0; uint32_t phase = 0;
            bool ok = true;
            int tr = 0;
            DPCLIP_TRACE_AT(0, 255);
            for (long u = u_begin; u < u_end && ok;) {
                const Seg w = segment_at(p, u, u_end, gj);
                if (w.layer < 0) { u += w.kb1 - w.kb0; continue; }
                const CUtensorMap* map_a = &maps.a[w.layer];
                const CUtensorMap* map_z = &maps.z[w.layer];
                const int mz = w.m0 + (int)rank * BM_CTA, na = w.n0 + (int)rank * BN_CTA;
                for (int kb = w.kb0; kb < w.kb1; ++kb) {
                    ok = mbar_wait(&empty[stage], phase ^ 1, abort_flag, p.status) &&
                         (!p.any_bias || mbar_wait(&zfree[stage], phase ^ 1, abort_flag, p.status));
                    if (!ok) break;
                    DPCLIP_TRACE_AT(0, tr); ++tr;
                    uint8_t* dst = smem + stage * STAGE_BYTES;
                    const int y = kb * BK;
                    mbar_arrive_expect_tx(&full[stage], STAGE_BYTES);
#pragma unroll
                    for (int c = 0; c < BM_CTA / 64; ++c)
                        tma_load_2d(dst + c * CHUNK_BYTES, map_z, &full[stage], mz + c * 64, y);
#pragma unroll
                    for (int c = 0; c < BN_CTA / 64; ++c)
                        tma_load_2d(dst + Z_BYTES + c * CHUNK_BYTES, map_a, &full[stage], na + c * 64, y);
                    if (++stage == STAGES) { stage = 0; phase ^= 1; }
                }
                u += w.kb1 - w.kb0;
            }
        }
    } else if (warp == 1) {
        // ------------------------------------------------ MMA issuer (rank 0 only)
        if (lane == 0 && rank == 0) {
            constexpr uint32_t idesc = make_idesc_bf16(256, BN, 1, 1);
            int stage = 0; uint32_t phase = 0; int it = 0;
            bool ok = true;
            int tr = 0;
            for (long u = u_begin; u < u_end && ok;) {
                const Seg w = segment_at(p, u, u_end, gj);
                if (w.layer < 0) { u += w.kb1 - w.kb0; continue; }
                ok = mbar_wait(acc_empty, (it & 1) ^ 1, abort_flag, p.status);
                if (!ok) break;
                tc_fence_after_sync();
                for (int kb = w.kb0; kb < w.kb1; ++kb) {
                    ok = mbar_wait(&ready[stage], phase, abort_flag, p.status);
                    if (!ok) break;
                    DPCLIP_TRACE_AT(2, tr); ++tr;
                    tc_fence_after_sync();
                    const uint32_t z_addr = smem_u32(smem + stage * STAGE_BYTES);
                    const uint32_t a_addr = z_addr + Z_BYTES;
#pragma unroll
                    for (int k4 = 0; k4 < BK / 16; ++k4) {
                        // MN-major, 128-byte swizzle: 64-column chunks CHUNK_BYTES apart (leading offset), 8-row
                        // groups 1024 bytes apart (stride offset); 16 rows = 2048 bytes.  The N-side descriptor
                        // names this CTA's 128 columns; the partner's 128 sit at the same offset in its memory.
                        const uint64_t db = make_smem_desc_sw128(a_addr + k4 * 2048, CHUNK_BYTES, 1024);
#pragma unroll
                        for (int h = 0; h < 2; ++h) {
                            const uint64_t da = make_smem_desc_sw128(z_addr + h * 2 * CHUNK_BYTES + k4 * 2048,
                                                                     CHUNK_BYTES, 1024);
                            mma_bf16_ss_pair(tmem_base + h * BN, da, db, idesc, (kb == w.kb0 && k4 == 0) ? 0u : 1u);
                        }
                    }
                    mma_commit_pair(&empty[stage], 3);          // frees the stage in both CTAs
                    if (++stage == STAGES) { stage = 0; phase ^= 1; }
                }
                if (!ok) break;
                mma_commit_pair(acc_full, 3);                   // both CTAs' epilogues may drain
                ++it;
                u += w.kb1 - w.kb0;
            }
        }
    } else if (warp < 2 + N_TRANSFORM_WARPS) {
        // ------------------------------------------------ transform (256 threads)
        // A half of a stage: 64 rows x 128 columns.  Thread t owns the 8 columns [8q, 8q + 8), q = t / 16, on
        // rows (t % 16) + 16 i.  Column chunk q sits at 16-byte slot (q % 8) ^ (row % 8) of its 128-byte row
        // (the TMA swizzle), the same slot for all rows of a thread.
        const int t = threadIdx.x - 64;
        const int q = t >> 4, rs = t & 15;
        const int box = q >> 3, lq = q & 7;
        const uint32_t off = box * CHUNK_BYTES + rs * 128 + ((lq ^ (rs & 7)) << 4);
        const uint32_t ready0 = mapa_shared(smem_u32(ready), 0);           // rank 0's `ready` barriers
        int stage = 0; uint32_t phase = 0;
        bool ok = true;
        int tr = 0;
        for (long u = u_begin; u < u_end && ok;) {
            const Seg w = segment_at(p, u, u_end, gj);
            if (w.layer < 0) { u += w.kb1 - w.kb0; continue; }
            const float* lclip = p.layer[w.layer].clip;
            for (int kb = w.kb0; kb < w.kb1; ++kb) {
                // the factors of this stage's rows are fetched BEFORE waiting for the tile, so the global-load
                // latency overlaps the wait instead of sitting between TMA and MMA
                const int blk0 = kb * BK;                              // rows [blk0, blk0 + BK)
                const int e_first = blk0 / p.T;
                const int rem0 = blk0 - e_first * p.T;
                const bool uniform = (rem0 + BK <= p.T) && (blk0 + BK <= p.R);   // one example, all rows exist
                constexpr int NR = BK / 16;
                float fr[NR];
                if (uniform) {
                    const float f = row_factor(p, lclip, e_first);     // one factor for the whole stage
#pragma unroll
                    for (int i = 0; i < NR; ++i) fr[i] = f;
                } else {
#pragma unroll
                    for (int i = 0; i < NR; ++i) {
                        const int rl = rs + 16 * i;
                        // past the last row TMA filled zeros; the factor only has to be finite there
                        fr[i] = blk0 + rl >= p.R ? 0.f : row_factor(p, lclip, e_first + (rem0 + rl) / p.T);
                    }
                }
                ok = mbar_wait(&full[stage], phase, abort_flag, p.status);
                if (!ok) break;
                if (t == 0) { DPCLIP_TRACE_AT(1, tr); ++tr; }
                uint8_t* at = smem + stage * STAGE_BYTES + Z_BYTES;
                // packed bf16 scaling: f = f_hi + f_lo (two bf16); a*f_lo is tiny, so the fused multiply-add
                // a*f_hi + (a*f_lo) rounds the product once
                auto scale8 = [](uint4& v, float f) {
                    const __nv_bfloat16 fh = __float2bfloat16_rn(f);
                    const __nv_bfloat16 fl = __float2bfloat16_rn(f - __bfloat162float(fh));
                    const __nv_bfloat162 fh2 = __halves2bfloat162(fh, fh), fl2 = __halves2bfloat162(fl, fl);
                    __nv_bfloat162* z2 = reinterpret_cast<__nv_bfloat162*>(&v);
#pragma unroll
                    for (int u2 = 0; u2 < 4; ++u2) z2[u2] = __hfma2(z2[u2], fh2, __hmul2(z2[u2], fl2));
                };
                bool any = false;
#pragma unroll
                for (int i = 0; i < NR; ++i) any = any || fr[i] != 1.f;
                if (any) {
                    // all loads before the first store: one shared-memory round trip per stage; rows whose
                    // factor is exactly 1 are left as they are
                    uint4 v[NR];
#pragma unroll
                    for (int i = 0; i < NR; ++i) v[i] = *reinterpret_cast<const uint4*>(at + off + i * 2048);
#pragma unroll
                    for (int i = 0; i < NR; ++i) {
                        if (fr[i] != 1.f) {
                            scale8(v[i], fr[i]);
                            *reinterpret_cast<uint4*>(at + off + i * 2048) = v[i];
                        }
                    }
                }
                fence_proxy_async_smem();
                __syncwarp();
                if (lane == 0) mbar_arrive_cluster(ready0 + stage * 8);
                if (t == 0) { DPCLIP_TRACE_AT(1, tr); ++tr; }
                if (++stage == STAGES) { stage = 0; phase ^= 1; }
            }
            u += w.kb1 - w.kb0;
        }
    } else {
        // ------------------------------------------------ epilogue (8 warps)
        // Warp w may touch tensor-memory lanes 32*(w % 4) .. +31.  Two warps share each lane quarter: group
        // g = 0/1 takes M sub-tile g (tensor-memory columns g * 256 ..).
        const int quarter = warp & 3;
        const int ew = warp - (2 + N_TRANSFORM_WARPS);
        const int h = ew >> 2;
        const uint32_t acc_empty0 = mapa_shared(smem_u32(acc_empty), 0);
        // bias sums: while the main loop runs these warps are idle, so THEY take the column sums
        // sum_rows c * zb of the Zb tile (read only, fp32), in parallel with the transform warps; same
        // thread-to-element map as the transform (thread t: 8 columns q of each 128-column half, rows rs + 16 i)
        const int t = threadIdx.x - 64 - 32 * N_TRANSFORM_WARPS;
        const int q = t >> 4, rs = t & 15;
        const uint32_t off = (q >> 3) * CHUNK_BYTES + rs * 128 + (((q & 7) ^ (rs & 7)) << 4);
        int stage = 0; uint32_t phase = 0;
        int it = 0;
        bool ok = true;
        for (long u = u_begin; u < u_end && ok;) {
            const Seg w = segment_at(p, u, u_end, gj);
            if (w.layer < 0) { u += w.kb1 - w.kb0; continue; }
            const Layer& y = p.layer[w.layer];
            const float* lclip = y.clip;
            if (p.any_bias) {
                float cs[2][8];
#pragma unroll
                for (int h2 = 0; h2 < 2; ++h2)
#pragma unroll
                    for (int j = 0; j < 8; ++j) cs[h2][j] = 0.f;
                for (int kb = w.kb0; kb < w.kb1; ++kb) {
                    // every n-tile of a row range sees the same Zb rows: stage kb's sums are taken by the n-tile
                    // with kb % tiles_n == tn (equal shares)
                    const bool bias_here = y.do_bias && (kb % y.tiles_n) == w.tn;
                    constexpr int NR = BK / 16;
                    float fr[NR];
                    if (bias_here) {
                        const int blk0 = kb * BK;
                        const int e_first = blk0 / p.T;
                        const int rem0 = blk0 - e_first * p.T;
                        const bool uniform = (rem0 + BK <= p.T) && (blk0 + BK <= p.R);
                        if (uniform) {
                            const float f = row_factor(p, lclip, e_first);
#pragma unroll
                            for (int i = 0; i < NR; ++i) fr[i] = f;
                        } else {
#pragma unroll
                            for (int i = 0; i < NR; ++i) {
                                const int rl = rs + 16 * i;
                                fr[i] = blk0 + rl >= p.R ? 0.f : row_factor(p, lclip, e_first + (rem0 + rl) / p.T);
                            }
                        }
                    }
                    ok = mbar_wait(&full[stage], phase, abort_flag, p.status);
                    if (!ok) break;
                    if (bias_here) {
                        const uint8_t* zt = smem + stage * STAGE_BYTES;
                        uint4 z[2][NR];
#pragma unroll
                        for (int h2 = 0; h2 < 2; ++h2)
#pragma unroll
                            for (int i = 0; i < NR; ++i)
                                z[h2][i] = *reinterpret_cast<const uint4*>(zt + h2 * 2 * CHUNK_BYTES + off + i * 2048);
#pragma unroll
                        for (int h2 = 0; h2 < 2; ++h2)
#pragma unroll
                            for (int i = 0; i < NR; ++i) {
                                const uint32_t wds[4] = {z[h2][i].x, z[h2][i].y, z[h2][i].z, z[h2][i].w};
#pragma unroll
                                for (int u2 = 0; u2 < 4; ++u2) {
                                    cs[h2][2 * u2] = fmaf(fr[i], __uint_as_float(wds[u2] << 16), cs[h2][2 * u2]);
                                    cs[h2][2 * u2 + 1] = fmaf(fr[i], __uint_as_float(wds[u2] & 0xFFFF0000u), cs[h2][2 * u2 + 1]);
                                }
                            }
                    }
                    __syncwarp();
                    if (lane == 0) mbar_arrive(&zfree[stage]);                    // this warp is done reading the stage
                    if (++stage == STAGES) { stage = 0; phase ^= 1; }
                }
                if (!ok) break;
                // finish the column sums over the 16 row-subsets (16 consecutive lanes); every segment writes its
                // 512 sums (zeros where it took none), so the reduce can add all segments of a tile row
#pragma unroll
                for (int h2 = 0; h2 < 2; ++h2)
#pragma unroll
                    for (int j = 0; j < 8; ++j) {
                        float c = cs[h2][j];
                        c += __shfl_xor_sync(0xFFFFFFFFu, c, 1);
                        c += __shfl_xor_sync(0xFFFFFFFFu, c, 2);
                        c += __shfl_xor_sync(0xFFFFFFFFu, c, 4);
                        c += __shfl_xor_sync(0xFFFFFFFFu, c, 8);
                        if (rs == 0 && DPCLIP_IN_RANGE(w.slot, p.n_segments, p.status))
                            p.bias_part[(size_t)w.slot * BM + (int)rank * BM_CTA + h2 * 128 + q * 8 + j] = c;
                    }
            }
            if (!mbar_wait(acc_full, it & 1, abort_flag, p.status)) break;
            if (ew == 0 && lane == 0) DPCLIP_TRACE_AT(3, 2 * it);
            tc_fence_after_sync();
            const uint32_t t_row = tmem_base + ((uint32_t)(quarter * 32) << 16) + h * BN;
            const int ml0 = (int)rank * BM_CTA + h * 128 + quarter * 32;     // first row of this warp in the pair tile
            float* seg = p.part + (size_t)w.slot * SEG_ELEMS;
#pragma unroll 1
            for (int c0 = 0; c0 < BN; c0 += 32) {
                uint32_t v[32];
                tmem_ld_32x32(t_row + c0, v);
                tmem_ld_wait();
                // Transpose the 32 x 32 block through shared memory so that every store covers 4 rows x 128
                // contiguous bytes instead of 32 rows x 16 bytes.
                float4* st = out_stage + ew * 256;
#pragma unroll
                for (int j = 0; j < 8; ++j)
                    st[lane * 8 + (j ^ (lane & 7))] =
                        make_float4(__uint_as_float(v[4 * j]), __uint_as_float(v[4 * j + 1]),
                                    __uint_as_float(v[4 * j + 2]), __uint_as_float(v[4 * j + 3]));
                __syncwarp();
                const int jj = lane & 7;
#pragma unroll
                for (int i = 0; i < 8; ++i) {
                    const int rr = 4 * i + (lane >> 3);
                    const float4 x = st[rr * 8 + (jj ^ (rr & 7))];
                    // the segment's partial tile (dense 512 x 256, no bounds: rows and columns past the layer's
                    // extent hold the zeros TMA filled in)
                    if (DPCLIP_IN_RANGE(w.slot, p.n_segments, p.status) && DPCLIP_IN_RANGE(ml0 + rr, BM, p.status))
                        *reinterpret_cast<float4*>(seg + (size_t)(ml0 + rr) * BN + c0 + 4 * jj) = x;
                }
                __syncwarp();
            }
            tc_fence_before_sync();
            __syncwarp();
            if (lane == 0) mbar_arrive_cluster(acc_empty0);
            if (ew == 0 && lane == 0) DPCLIP_TRACE_AT(3, 2 * it + 1);
            ++it;
            u += w.kb1 - w.kb0;
        }
    }

    // ---------------------------------------------------- teardown
    if (*abort_flag) {
        for (int i = 0; i < 64; ++i) __nanosleep(1000);
    }
    tc_fence_before_sync();
    cluster_sync_all();             // nobody frees tensor memory or exits while its partner may still signal it
    if (warp == 1) { tc_fence_after_sync(); tmem_dealloc_pair(tmem_base, 512); }
}

// ---------------------------------------------------------------------------
// Second stage: every output element = the fixed-order sum of its tile's segments (+ Philox noise), every bias =
// the sum over the n-tiles and segments of its tile row.
// ---------------------------------------------------------------------------
__global__ void __launch_bounds__(256, 6)            // six CTAs per SM: the launch is one wave of 6 x SMs
reduce_segments_kernel(const __grid_constant__ ztp::Params p) {
    using namespace ztp;
    // One wave of CTAs over the 4-row x 256-column blocks of every tile of every layer, one float4 per thread and
    // block.  A tile's layer and segment range come from the host's tables (working the range out here cost six
    // 64-bit divisions per block).  A thread issues the loads of up to four segments before the first add and draws
    // its noise while they are in flight: with one load in flight per thread the kernel was bound by the latency of
    // its serial loads; what binds it now is instruction issue (the Philox rounds and Box-Muller of every float4).
    constexpr int ROWS = 4, SG = 4;
    constexpr int ROW_BLOCKS = BM / ROWS;
    const int n_blocks = p.G * ROW_BLOCKS;
    const size_t seg_stride = (size_t)p.W * SEG_ELEMS;
    const int c4 = (threadIdx.x & 63) << 2, r = threadIdx.x >> 6;
    for (int blk = blockIdx.x; blk < n_blocks; blk += gridDim.x) {
        const int t = blk / ROW_BLOCKS, rb = blk - t * ROW_BLOCKS;
        const Layer& y = p.layer[p.tile_layer[t]];
        const int tile = t - y.tile_base;
        const int tm = tile / y.tiles_n, tn = tile - tm * y.tiles_n;
        const int m = tm * BM + rb * ROWS + r, n = tn * BN + c4;
        if (m >= y.d_out || n >= y.d_in) continue;
        const int first = p.seg_first[t], n_seg = p.seg_count[t];
        if (!DPCLIP_IN_RANGE(first + (long)(n_seg - 1) * p.W, p.n_segments, p.status) || n_seg < 1) continue;
        const float* src = p.part + (size_t)first * SEG_ELEMS + (size_t)(rb * ROWS + r) * BN + c4;
        float4 v[SG];
#pragma unroll
        for (int k = 0; k < SG; ++k)
            v[k] = k < n_seg ? __ldcs(reinterpret_cast<const float4*>(src + (size_t)k * seg_stride))
                             : make_float4(0.f, 0.f, 0.f, 0.f);
        float z0 = 0.f, z1 = 0.f, z2 = 0.f, z3 = 0.f;
        if (p.noise_scale > 0.f) {
            const size_t qd = ((size_t)m * y.d_in + n) >> 2;
            PhiloxBlock b = philox_block((uint32_t)qd, (uint32_t)(qd >> 32), y.sw0, y.sw1, p.k0, p.k1);
            box_muller(b.v[0], b.v[1], z0, z1);
            box_muller(b.v[2], b.v[3], z2, z3);
        }
        float4 acc = v[0];                                                  // segment order
#pragma unroll
        for (int k = 1; k < SG; ++k) { acc.x += v[k].x; acc.y += v[k].y; acc.z += v[k].z; acc.w += v[k].w; }
        for (int sb = SG; sb < n_seg; sb += SG) {                           // tiles cut into more than four runs
#pragma unroll
            for (int k = 0; k < SG; ++k)
                v[k] = sb + k < n_seg ? __ldcs(reinterpret_cast<const float4*>(src + (size_t)(sb + k) * seg_stride))
                                      : make_float4(0.f, 0.f, 0.f, 0.f);
#pragma unroll
            for (int k = 0; k < SG; ++k) { acc.x += v[k].x; acc.y += v[k].y; acc.z += v[k].z; acc.w += v[k].w; }
        }
        if (p.noise_scale > 0.f) {
            acc.x = fmaf(p.noise_scale, z0, acc.x); acc.y = fmaf(p.noise_scale, z1, acc.y);
            acc.z = fmaf(p.noise_scale, z2, acc.z); acc.w = fmaf(p.noise_scale, z3, acc.w);
        }
        float* dst = y.gW + (size_t)m * y.ldg + n;
        if (y.vec_ok && n + 4 <= y.d_in) {
            *reinterpret_cast<float4*>(dst) = acc;
        } else {
            const float xs[4] = {acc.x, acc.y, acc.z, acc.w};
            for (int q = 0; q < 4; ++q)
                if (n + q < y.d_in) dst[q] = xs[q];
        }
    }
    if (p.any_bias) {
        // bias: one warp per output, the outputs of all layers with a bias numbered in one sequence (so every warp
        // of the grid has at most one or two of them).  Its lanes take eight n-tiles x four segments of the tile row
        // at a time: the partial sums of a row are usually fetched by one load per lane (a serial walk over layers
        // and n-tiles left a tail of several microseconds at the end of the kernel).
        const int lane = threadIdx.x & 31;
        int total = 0;
        for (int l = 0; l < p.n_layers; ++l) total += (p.layer[l].do_bias && p.layer[l].gb) ? p.layer[l].d_out : 0;
        for (int g = (blockIdx.x * blockDim.x + threadIdx.x) >> 5; g < total; g += (gridDim.x * blockDim.x) >> 5) {
            int l = 0, m = g;
            for (; l < p.n_layers; ++l) {
                const int rows = (p.layer[l].do_bias && p.layer[l].gb) ? p.layer[l].d_out : 0;
                if (m < rows) break;
                m -= rows;
            }
            const Layer& y = p.layer[l];
            const int tm = m / BM;
            float acc = 0.f;
            for (int tn = lane >> 2; tn < y.tiles_n; tn += 8) {
                const int t = y.tile_base + tm * y.tiles_n + tn;
                const int first = p.seg_first[t], n_seg = p.seg_count[t];
                for (int k = lane & 3; k < n_seg; k += 4)
                    acc += p.bias_part[(size_t)(first + (long)k * p.W) * BM + (m - tm * BM)];
            }
            acc = warp_sum(acc);
            if (lane != 0) continue;
            if (p.noise_scale > 0.f) {
                PhiloxBlock b = philox_block((uint32_t)(m >> 2), 0u, y.sb0, y.sb1, p.k0, p.k1);
                float z[4];
                box_muller(b.v[0], b.v[1], z[0], z[1]);
                box_muller(b.v[2], b.v[3], z[2], z[3]);
                acc = fmaf(p.noise_scale, z[m & 3], acc);
            }
            y.gb[m] = acc;
        }
    }
}

}  // namespace tc
}  // namespace dpclip
