// tcgen05 / TMEM / TMA kernels for bf16 layers.
//
//   gram_norm_kernel : per-example squared norms by the Gram identity
//       ||sum_t zb_t (x) a_t||_F^2 = sum_{t,s} (a_t . a_s)(zb_t . zb_s)
//     Both Gram factors of a 128 x 256 block of (t, s) pairs (one row block
//     against two column blocks) are accumulated in tensor memory (A A^T in
//     columns 0..255, Zb Zb^T in 256..511, fp32) from K-major operand tiles
//     fetched by TMA; the epilogue multiplies the two blocks element-wise and
//     reduces, so no Gram matrix reaches HBM.  One CTA walks all blocks of an
//     example, so re-reads of a tile come from L2.  Rows are
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
//                  the epilogue writes the CTA's partial tile to the workspace
//                  (reduce_partials_kernel adds the tiles in a fixed order), or
//                  straight to gW when a tile has a single row slice.
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

// Developer-only timeline (compiled in with -DDPCLIP_TRACE; never in the shipped library).
#ifdef DPCLIP_TRACE
__device__ unsigned long long g_trace[148][4][256];
#define DPCLIP_TRACE_AT(role, idx) do { if ((idx) < 256) g_trace[blockIdx.x][role][idx] = global_ns(); } while (0)
#else
#define DPCLIP_TRACE_AT(role, idx) do { } while (0)
#endif

// ===========================================================================
// Gram kernel
// ===========================================================================
namespace gram {
constexpr int BM = 128;                       // rows per block (t and s)
constexpr int BK = 64;                        // features per stage = one 128-byte swizzle row
constexpr int TILE_BYTES = BM * BK * 2;       // 16 KB: 128 rows x 64 features
// A stage holds the row block's tile and up to two column blocks' tiles.  When every item sits on
// the diagonal (examples of at most 256 rows, T % 128 == 0) the row block IS the first column block,
// so stages shrink to two tiles and six of them fit: more bytes in flight per SM, which is what
// bounds a kernel whose tiles are used once.
template <bool DIAG_ONLY> struct Cfg {
    static constexpr int TILES = DIAG_ONLY ? 2 : 3;
    static constexpr int STAGE_BYTES = TILES * TILE_BYTES;
    static constexpr int STAGES = DIAG_ONLY ? 6 : 4;
};
constexpr int N_EPILOGUE_WARPS = 8;
constexpr int THREADS = 64 + 32 * N_EPILOGUE_WARPS;   // warp 0 TMA, warp 1 MMA, warps 2..9 epilogue
constexpr int SMEM_BYTES = 4 * 3 * TILE_BYTES + 1024 /*alignment slack*/ + 512 /*barriers, queues, warp sums*/;   // = 6 * 2 tiles

constexpr int MAX_LAYERS = 8;                 // layers one launch can take

struct Params {            // one layer
    int R, T, d_in, d_out, has_bias;
    int n_groups;          // dense (T % 128 == 0): examples; otherwise: 128-row blocks
    int dense, q;          // q = T / 128 blocks per example in the dense case
    float* sq;
};

// One launch: the groups of up to MAX_LAYERS layers, dealt to the CTAs in one sequence (layer 0's groups
// first).  With one example per CTA a single layer of a small batch is a latency chain (set-up, first
// load, the second row block and both epilogues are all exposed); several layers in one launch give every
// CTA a queue of items, so loads of the next item run under the MMAs and epilogues of the current one.
// Clip factors in the tail of a norm launch that produces EVERY row of sq[L][B] (the text after Eq.
// "weighted_loss" and Eq. "per_example_weight": n_i = sqrt(sum_l sq[l][i]), c_i = min(1, C / n_i)): the CTA
// that finishes last computes them, so the step needs no factors launch between its norms and its clipped
// sums.  Same arithmetic, in the same order, as factors_kernel.
struct FactorsTail {
    const float* sq; int L; long ld; int B; float C;
    float* clip; float* norms;           // clip == NULL: no tail
    unsigned int* done;                  // CTAs finished so far (workspace header; back at zero after the launch)
};

struct Launch {
    CUtensorMap map_a[MAX_LAYERS], map_z[MAX_LAYERS];
    Params layer[MAX_LAYERS];
    int group_begin[MAX_LAYERS + 1];
    int L, total_groups;
    int* status;
    unsigned int* work_counter;    // gram_norm_q2_kernel: items are handed out in order from this counter
    FactorsTail tail;
};

// Called by every thread of a CTA after its last atomic into sq has been issued.
__device__ __forceinline__ void factors_tail(const FactorsTail& t) {
    if (!t.clip) return;
    __shared__ unsigned int s_prev;
    __threadfence();                                   // this thread's atomics on sq before the CTA's count
    __syncthreads();
    if (threadIdx.x == 0) s_prev = atomicAdd(t.done, 1u);
    __syncthreads();
    if (s_prev != gridDim.x - 1) return;               // not the last CTA
    __threadfence();
    for (int i = threadIdx.x; i < t.B; i += blockDim.x) {
        float s = 0.f;
        for (int l = 0; l < t.L; ++l) s += __ldcg(t.sq + (size_t)l * t.ld + i);      // L2: where the atomics landed
        const float n = sqrtf(s);
        float c = 1.0f;
        if (n > t.C) c = t.C / n;                      // tie and zero norm stay exactly 1
        t.clip[i] = c;
        if (t.norms) t.norms[i] = n;
    }
    if (threadIdx.x == 0) *t.done = 0u;                // ready for the next launch
}

// layer of group g (group_begin is ascending; L is small)
__device__ __forceinline__ int layer_of(const Launch& q, int g) {
    int l = 0;
#pragma unroll 1
    while (l + 1 < q.L && g >= q.group_begin[l + 1]) ++l;
    return l;
}

// One unit of MMA work: row block rb against column blocks cb .. cb + ncb - 1 (ncb = 1 or 2).
struct Sub { int rb, cb, ncb; };

// The sub-items of group g, in a fixed order that every warp role walks identically.
// Row block rb pairs with column blocks rb .. cb_max(rb) (those that still hold rows of an example
// that has rows in rb), taken two at a time so that one 128 x 256 MMA covers two of them.
// In the dense case the row blocks of an example are walked from the LAST to the first: row block rb needs
// the column blocks rb .. q-1, so every pass then fetches exactly one block that has not been read before
// (its own) and re-reads the others from L2.  Walking upwards, the first pass streams the whole example
// from HBM and the later ones run out of L2; CTAs that start together then alternate in lockstep between
// a phase that saturates HBM and one that leaves it idle (measured: 23 us per 512 KB example instead of the
// 12.5 us its bytes take).
struct SubIter {
    int rb, rb_first, rb_last, cb, cb_max;
    __device__ __forceinline__ static int cbmax(const Params& p, int rb) {
        const long last_row = min((long)rb * BM + BM - 1, (long)p.R - 1);
        const long e_last = last_row / p.T;
        return (int)(min((e_last + 1) * p.T - 1, (long)p.R - 1) / BM);
    }
    __device__ __forceinline__ SubIter(const Params& p, int g) {
        if (p.dense) { rb_first = g * p.q; rb_last = rb_first + p.q - 1; } else { rb_first = g; rb_last = g; }
        rb = rb_last;
        cb = rb; cb_max = cbmax(p, rb);
    }
    __device__ __forceinline__ bool next(const Params& p, Sub& s) {
        if (rb < rb_first) return false;
        s.rb = rb; s.cb = cb; s.ncb = cb + 1 <= cb_max ? 2 : 1;
        cb += 2;
        if (cb > cb_max) { --rb; if (rb >= rb_first) { cb = rb; cb_max = cbmax(p, rb); } }
        return true;
    }
};
}  // namespace gram

template <bool DIAG_ONLY>
__global__ void __launch_bounds__(gram::THREADS, 1)
gram_norm_kernel(const __grid_constant__ gram::Launch q) {
    using namespace gram;
    constexpr int STAGES = Cfg<DIAG_ONLY>::STAGES, STAGE_BYTES = Cfg<DIAG_ONLY>::STAGE_BYTES;
    // offset of the first column block's tile inside a stage (the row block's own tile comes first
    // only when stages have room for it)
    constexpr int B_OFF = DIAG_ONLY ? 0 : TILE_BYTES;
    extern __shared__ uint8_t smem_raw[];
    uint8_t* smem = smem_raw + ((1024u - (smem_u32(smem_raw) & 1023u)) & 1023u);   // 1024-byte aligned; an offset from the array keeps the accesses in the shared state space
    uint64_t* full = reinterpret_cast<uint64_t*>(smem + STAGES * STAGE_BYTES);
    uint64_t* empty = full + STAGES;
    uint64_t* acc_full = empty + STAGES;
    uint64_t* acc_empty = acc_full + 1;
    uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(acc_empty + 1);
    volatile int* abort_flag = reinterpret_cast<volatile int*>(tmem_slot + 1);

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    if (threadIdx.x == 0) {
        for (int s = 0; s < STAGES; ++s) { mbar_init(&full[s], 1); mbar_init(&empty[s], 1); }
        mbar_init(acc_full, 1); mbar_init(acc_empty, N_EPILOGUE_WARPS);
        *abort_flag = 0;
        mbar_fence_init();
        for (int l = 0; l < q.L; ++l) { tma_prefetch_desc(&q.map_a[l]); tma_prefetch_desc(&q.map_z[l]); }
    }
    if (warp == 1) { tmem_alloc(tmem_slot, 512); tmem_relinquish(); }
    tc_fence_before_sync();
    __syncthreads();
    tc_fence_after_sync();
    const uint32_t tmem_base = *tmem_slot;      // A A^T in columns 0..255, Zb Zb^T in 256..511

    if (warp == 0) {
        // ------------------------------------------------ TMA producer
        if (lane == 0) {
            int stage = 0; uint32_t phase = 0;
            bool ok = true;
            int tr = 0;
            DPCLIP_TRACE_AT(0, 255);
            for (int g = blockIdx.x; g < q.total_groups && ok; g += gridDim.x) {
                const int l = layer_of(q, g);
                const Params& p = q.layer[l];
                const int nk_a = (p.d_in + BK - 1) / BK, nk_z = (p.d_out + BK - 1) / BK;
                SubIter it(p, g - q.group_begin[l]);
                Sub s;
                while (ok && it.next(p, s)) {
                    const bool diag = s.rb == s.cb;
                    const uint32_t bytes = TILE_BYTES * (s.ncb + (diag ? 0 : 1));
                    const int nk = nk_a + nk_z;
                    for (int kb = 0; kb < nk; ++kb) {
                        const CUtensorMap* map = kb < nk_a ? &q.map_a[l] : &q.map_z[l];
                        const int x = (kb < nk_a ? kb : kb - nk_a) * BK;
                        ok = mbar_wait(&empty[stage], phase ^ 1, abort_flag, q.status);
                        if (!ok) break;
                        DPCLIP_TRACE_AT(0, tr); ++tr;
                        uint8_t* dst = smem + stage * STAGE_BYTES;
                        mbar_arrive_expect_tx(&full[stage], bytes);
                        if (!DIAG_ONLY && !diag) tma_load_2d(dst, map, &full[stage], x, s.rb * BM);
                        tma_load_2d(dst + B_OFF, map, &full[stage], x, s.cb * BM);
                        if (s.ncb == 2) tma_load_2d(dst + B_OFF + TILE_BYTES, map, &full[stage], x, (s.cb + 1) * BM);
                        if (++stage == STAGES) { stage = 0; phase ^= 1; }
                    }
                }
            }
        }
    } else if (warp == 1) {
        // ------------------------------------------------ MMA issuer
        if (lane == 0) {
            int stage = 0; uint32_t phase = 0; uint32_t acc_phase = 0;
            bool ok = true;
            int tr = 0;
            for (int g = blockIdx.x; g < q.total_groups && ok; g += gridDim.x) {
                const int l = layer_of(q, g);
                const Params& p = q.layer[l];
                const int nk_a = (p.d_in + BK - 1) / BK, nk_z = (p.d_out + BK - 1) / BK;
                SubIter it(p, g - q.group_begin[l]);
                Sub s;
                while (ok && it.next(p, s)) {
                    const uint32_t idesc = make_idesc_bf16(BM, BM * s.ncb, 0, 0);
                    ok = mbar_wait(acc_empty, acc_phase ^ 1, abort_flag, q.status);
                    if (!ok) break;
                    tc_fence_after_sync();
                    for (int kb = 0; kb < nk_a + nk_z; ++kb) {
                        const bool is_a = kb < nk_a;
                        const uint32_t d_tmem = tmem_base + (is_a ? 0 : 256);
                        const bool first = is_a ? kb == 0 : kb == nk_a;
                        ok = mbar_wait(&full[stage], phase, abort_flag, q.status);
                        if (!ok) break;
                        DPCLIP_TRACE_AT(2, tr); ++tr;
                        tc_fence_after_sync();
                        const uint32_t b_addr = smem_u32(smem + stage * STAGE_BYTES) + B_OFF;
                        const uint32_t a_addr = (DIAG_ONLY || s.rb == s.cb) ? b_addr : b_addr - TILE_BYTES;
#pragma unroll
                        for (int k4 = 0; k4 < BK / 16; ++k4) {
                            // K-major, 128-byte swizzle: 8-row groups 1024 bytes apart; 16 features = 32 bytes.
                            // The two column blocks are contiguous, so N = 256 simply runs on.
                            const uint64_t da = make_smem_desc_sw128(a_addr + k4 * 32, 16, 1024);
                            const uint64_t db = make_smem_desc_sw128(b_addr + k4 * 32, 16, 1024);
                            mma_bf16_ss(d_tmem, da, db, idesc, (first && k4 == 0) ? 0u : 1u);
                        }
                        mma_commit(&empty[stage]);
                        if (++stage == STAGES) { stage = 0; phase ^= 1; }
                    }
                    if (!ok) break;
                    mma_commit(acc_full);
                    acc_phase ^= 1;
                }
            }
        }
    } else {
        // ------------------------------------------------ epilogue (warps 2..9)
        // warp w reads tensor-memory lanes 32*(w % 4)..+31; the two warps of a lane quarter take
        // the two column blocks of the item.
        const int quarter = warp & 3;
        const int half = (warp - 2) >> 2;
        const int row_local = quarter * 32 + lane;
        uint32_t acc_phase = 0;
        bool ok = true;
        int etr = 0;
        for (int g = blockIdx.x; g < q.total_groups && ok; g += gridDim.x) {
            const int l = layer_of(q, g);
            const Params& p = q.layer[l];
            SubIter it(p, g - q.group_begin[l]);
            Sub s;
            while (it.next(p, s)) {
                ok = mbar_wait(acc_full, acc_phase, abort_flag, q.status);
                if (!ok) break;
                if (threadIdx.x == 64) { DPCLIP_TRACE_AT(3, etr); ++etr; }
                acc_phase ^= 1;
                tc_fence_after_sync();
                float val = 0.f;
                long e = 0;
                bool valid = false;
                if (half < s.ncb) {
                    const int cbk = s.cb + half;                 // this warp's column block
                    const long r = (long)s.rb * BM + row_local;
                    valid = r < p.R;
                    e = valid ? r / p.T : 0;
                    // columns of the block that belong to the same example as row r
                    int lo = (int)(max(e * p.T, (long)cbk * BM) - (long)cbk * BM);
                    int hi = (int)(min(min((e + 1) * p.T, (long)p.R), (long)cbk * BM + BM) - (long)cbk * BM);
                    if (!valid) { lo = 0; hi = 0; }
                    float sa = 0.f, sb = 0.f;
                    const uint32_t t_row = tmem_base + ((uint32_t)(quarter * 32) << 16) + half * BM;
#pragma unroll 1
                    for (int c0 = 0; c0 < BM; c0 += 32) {
                        uint32_t va[32], vz[32];
                        tmem_ld_32x32(t_row + c0, va);
                        tmem_ld_32x32(t_row + 256 + c0, vz);
                        tmem_ld_wait();
                        if (lo <= c0 && c0 + 32 <= hi) {             // whole chunk inside the example
#pragma unroll
                            for (int j = 0; j < 32; ++j) {
                                const float z = __uint_as_float(vz[j]);
                                sa = fmaf(__uint_as_float(va[j]), z, sa);
                                sb += z;
                            }
                        } else if (c0 < hi && c0 + 32 > lo) {
#pragma unroll
                            for (int j = 0; j < 32; ++j) {
                                const int col = c0 + j;
                                if (col >= lo && col < hi) {
                                    const float z = __uint_as_float(vz[j]);
                                    sa = fmaf(__uint_as_float(va[j]), z, sa);
                                    sb += z;
                                }
                            }
                        }
                    }
                    // blocks above the diagonal stand for their mirror image too
                    val = (cbk > s.rb ? 2.f : 1.f) * (sa + (p.has_bias ? sb : 0.f));
                    if (hi <= lo) valid = false;
                }
                tc_fence_before_sync();
                __syncwarp();
                if (lane == 0) mbar_arrive(acc_empty);
                if (threadIdx.x == 64) { DPCLIP_TRACE_AT(3, etr); ++etr; }
                const long e0 = __shfl_sync(0xFFFFFFFFu, e, 0);
                const bool uniform = __all_sync(0xFFFFFFFFu, valid && e == e0);
                if (uniform) {
                    val = warp_sum(val);
                    if (lane == 0) atomicAdd(p.sq + e0, val);
                } else if (valid) {
                    atomicAdd(p.sq + e, val);
                }
            }
        }
    }

    // ---------------------------------------------------- teardown
    if (*abort_flag) {                                      // let copies in flight land before the CTA exits
        for (int i = 0; i < 64; ++i) __nanosleep(1000);
    }
    tc_fence_before_sync();
    __syncthreads();
    if (warp == 1) { tc_fence_after_sync(); tmem_dealloc(tmem_base, 512); }
    factors_tail(q.tail);
}

// ---------------------------------------------------------------------------
// Gram kernel for examples of exactly two 128-row blocks (T = 256), every layer of the launch.
//
// The generic kernel walks such an example as two passes (row block 1 against itself, then row block 0
// against both), and the second pass re-reads half of the example.  With one example per SM in flight, 148
// examples' worth of other data passes through L2 between the two reads, so for wide layers the re-read
// comes from HBM again (measured: 1.5x the algorithmic DRAM traffic).  Here each K-chunk of the WIDER
// operand X is fetched once and feeds both its products at once:
//     P1  X rows 0..255  ->  G^X_0  = X_0 [X_0; X_1]^T  (tensor-memory columns   0..255)
//                            G^X_11 = X_1 X_1^T         (columns 256..383)
//     P2  Y rows 128..255 -> G^Y_11                     (columns 384..511)   epilogue E1: <G^X_11, G^Y_11>
//     P3  Y rows 0..255  ->  G^Y_0                      (columns 256..511)   epilogue E0: <G^X_0, G^Y_0>,
//                                                                            block (0,1) counted twice
// Only the narrower operand's second half is read twice, a few hundred KB apart (an L2 hit).  All 512
// columns are in use, so E1 must finish before P3 starts and E0 before the next example's P1.
//
// An example belongs to one CTA, so its squared norm is STORED, not accumulated: the eight epilogue warps leave
// their sums in shared memory and the first of them adds these in a fixed order.  The row of sq needs no
// clearing before the launch and the result does not depend on the order of atomics.
// ---------------------------------------------------------------------------
__global__ void __launch_bounds__(gram::THREADS, 1)
gram_norm_q2_kernel(const __grid_constant__ gram::Launch q) {
    using namespace gram;
    constexpr int STAGES = 6, STAGE_BYTES = 2 * TILE_BYTES;
    constexpr int SCHED = 4;                               // depth of the item queue
    extern __shared__ uint8_t smem_raw[];
    uint8_t* smem = smem_raw + ((1024u - (smem_u32(smem_raw) & 1023u)) & 1023u);   // 1024-byte aligned; an offset from the array keeps the accesses in the shared state space
    uint64_t* full = reinterpret_cast<uint64_t*>(smem + STAGES * STAGE_BYTES);
    uint64_t* empty = full + STAGES;
    uint64_t* acc_full = empty + STAGES;
    uint64_t* acc_empty = acc_full + 1;
    uint64_t* sched_full = acc_empty + 1;                  // item queue: producer -> MMA issuer and epilogue warps
    uint64_t* sched_empty = sched_full + SCHED;
    volatile int* sched_item = reinterpret_cast<volatile int*>(sched_empty + SCHED);
    uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(const_cast<int*>(sched_item) + SCHED);
    volatile int* abort_flag = reinterpret_cast<volatile int*>(tmem_slot + 1);
    // barriers and queue end 200 bytes into their area; the next 8-byte boundary is three ints past the flag's address
    static_assert((2 * STAGES + 2 + 2 * SCHED) * 8 + SCHED * 4 + 4 == 196, "offset of the abort flag");
    uint64_t* sums_full = reinterpret_cast<uint64_t*>(const_cast<int*>(abort_flag) + 3);   // [2]: warp sums of an example are in
    volatile float* sums = reinterpret_cast<volatile float*>(sums_full + 2);               // [2][N_EPILOGUE_WARPS]
    static_assert(STAGES * STAGE_BYTES + 208 + 16 + 2 * N_EPILOGUE_WARPS * 4 + 1024 <= SMEM_BYTES, "shared memory layout");

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    if (threadIdx.x == 0) {
        for (int s = 0; s < STAGES; ++s) { mbar_init(&full[s], 1); mbar_init(&empty[s], 1); }
        mbar_init(acc_full, 1); mbar_init(acc_empty, N_EPILOGUE_WARPS);
        for (int s = 0; s < SCHED; ++s) { mbar_init(&sched_full[s], 1); mbar_init(&sched_empty[s], 1 + N_EPILOGUE_WARPS); }
        mbar_init(&sums_full[0], N_EPILOGUE_WARPS); mbar_init(&sums_full[1], N_EPILOGUE_WARPS);
        *abort_flag = 0;
        mbar_fence_init();
        for (int l = 0; l < q.L; ++l) { tma_prefetch_desc(&q.map_a[l]); tma_prefetch_desc(&q.map_z[l]); }
    }
    if (warp == 1) { tmem_alloc(tmem_slot, 512); tmem_relinquish(); }
    tc_fence_before_sync();
    __syncthreads();
    tc_fence_after_sync();
    const uint32_t tmem_base = *tmem_slot;
    griddep_launch_dependents();    // the clipped-sum launch that follows may place its CTAs as SMs fall idle

    if (warp == 0) {
        // ------------------------------------------------ TMA producer
        if (lane == 0) {
            int stage = 0; uint32_t phase = 0;
            int slot = 0; uint32_t sphase = 0;
            bool ok = true;
            [[maybe_unused]] int tr = 0;
            DPCLIP_TRACE_AT(0, 255);
            // Items (layer-major, widest layers first) are taken in order from a counter shared by the CTAs,
            // so a CTA that drew wide examples simply draws fewer of them.  Every CTA draws until it sees a
            // value past the end, exactly once: after total + grid draws the counter has wrapped to zero,
            // ready for the next launch.  The next item is drawn before the loads of the current one are
            // issued, and published to the other roles through a small queue in shared memory.
            const unsigned int wrap = (unsigned int)q.total_groups + gridDim.x - 1;
            int g_next = (int)atomicInc(q.work_counter, wrap);
            while (ok) {
                const int g = g_next < q.total_groups ? g_next : -1;
                if (g >= 0) g_next = (int)atomicInc(q.work_counter, wrap);
                ok = mbar_wait(&sched_empty[slot], sphase ^ 1, abort_flag, q.status);
                if (!ok) break;
                sched_item[slot] = g;
                mbar_arrive(&sched_full[slot]);
                if (++slot == SCHED) { slot = 0; sphase ^= 1; }
                if (g < 0) break;
                const int l = layer_of(q, g);
                const Params& p = q.layer[l];
                const bool x_is_z = p.d_out > p.d_in;
                const CUtensorMap* map_x = x_is_z ? &q.map_z[l] : &q.map_a[l];
                const CUtensorMap* map_y = x_is_z ? &q.map_a[l] : &q.map_z[l];
                const int nk_x = ((x_is_z ? p.d_out : p.d_in) + BK - 1) / BK;
                const int nk_y = ((x_is_z ? p.d_in : p.d_out) + BK - 1) / BK;
                const int r0 = (g - q.group_begin[l]) * 2 * BM;
                for (int kb = 0; kb < nk_x + 2 * nk_y && ok; ++kb) {
                    // P1: both blocks of X; P2: block 1 of Y; P3: both blocks of Y
                    const bool p1 = kb < nk_x, p2 = !p1 && kb < nk_x + nk_y;
                    const CUtensorMap* map = p1 ? map_x : map_y;
                    const int x = (p1 ? kb : (p2 ? kb - nk_x : kb - nk_x - nk_y)) * BK;
                    ok = mbar_wait(&empty[stage], phase ^ 1, abort_flag, q.status);
                    if (!ok) break;
                    DPCLIP_TRACE_AT(0, tr); ++tr;
                    uint8_t* dst = smem + stage * STAGE_BYTES;
                    mbar_arrive_expect_tx(&full[stage], p2 ? TILE_BYTES : 2 * TILE_BYTES);
                    if (p2) {
                        tma_load_2d(dst, map, &full[stage], x, r0 + BM);
                    } else {
                        tma_load_2d(dst, map, &full[stage], x, r0);
                        tma_load_2d(dst + TILE_BYTES, map, &full[stage], x, r0 + BM);
                    }
                    if (++stage == STAGES) { stage = 0; phase ^= 1; }
                }
            }
        }
    } else if (warp == 1) {
        // ------------------------------------------------ MMA issuer
        if (lane == 0) {
            constexpr uint32_t idesc256 = make_idesc_bf16(BM, 2 * BM, 0, 0), idesc128 = make_idesc_bf16(BM, BM, 0, 0);
            int stage = 0; uint32_t phase = 0; uint32_t acc_phase = 0;
            int slot = 0; uint32_t sphase = 0;
            bool ok = true;
            [[maybe_unused]] int tr = 0;
            while (ok) {
                ok = mbar_wait(&sched_full[slot], sphase, abort_flag, q.status);
                if (!ok) break;
                const int g = sched_item[slot];
                mbar_arrive(&sched_empty[slot]);
                if (++slot == SCHED) { slot = 0; sphase ^= 1; }
                if (g < 0) break;
                const int l = layer_of(q, g);
                const Params& p = q.layer[l];
                const bool x_is_z = p.d_out > p.d_in;
                const int nk_x = ((x_is_z ? p.d_out : p.d_in) + BK - 1) / BK;
                const int nk_y = ((x_is_z ? p.d_in : p.d_out) + BK - 1) / BK;
                // the previous example's last epilogue has read every column
                ok = mbar_wait(acc_empty, acc_phase ^ 1, abort_flag, q.status);
                if (!ok) break;
                tc_fence_after_sync();
                for (int kb = 0; kb < nk_x + 2 * nk_y; ++kb) {
                    const bool p1 = kb < nk_x, p2 = !p1 && kb < nk_x + nk_y;
                    if (kb == nk_x + nk_y) {
                        // P2 is complete: hand G^X_11, G^Y_11 to the epilogue and wait until it has read them
                        // (P3 overwrites their columns)
                        mma_commit(acc_full);
                        acc_phase ^= 1;
                        ok = mbar_wait(acc_empty, acc_phase ^ 1, abort_flag, q.status);
                        if (!ok) break;
                        tc_fence_after_sync();
                    }
                    ok = mbar_wait(&full[stage], phase, abort_flag, q.status);
                    if (!ok) break;
                    DPCLIP_TRACE_AT(2, tr); ++tr;
                    tc_fence_after_sync();
                    const uint32_t t0 = smem_u32(smem + stage * STAGE_BYTES), t1 = t0 + TILE_BYTES;
                    const bool first = p1 ? kb == 0 : (p2 ? kb == nk_x : kb == nk_x + nk_y);
#pragma unroll
                    for (int k4 = 0; k4 < BK / 16; ++k4) {
                        // K-major, 128-byte swizzle: 8-row groups 1024 bytes apart; 16 features = 32 bytes.
                        // The two row blocks of a stage are contiguous, so N = 256 simply runs on.
                        const uint32_t acc = (first && k4 == 0) ? 0u : 1u;
                        const uint64_t d0 = make_smem_desc_sw128(t0 + k4 * 32, 16, 1024);
                        if (p1) {
                            const uint64_t d1 = make_smem_desc_sw128(t1 + k4 * 32, 16, 1024);
                            mma_bf16_ss(tmem_base, d0, d0, idesc256, acc);               // G^X_0
                            mma_bf16_ss(tmem_base + 256, d1, d1, idesc128, acc);         // G^X_11
                        } else if (p2) {
                            mma_bf16_ss(tmem_base + 384, d0, d0, idesc128, acc);         // G^Y_11 (the stage holds block 1)
                        } else {
                            mma_bf16_ss(tmem_base + 256, d0, d0, idesc256, acc);         // G^Y_0
                        }
                    }
                    mma_commit(&empty[stage]);
                    if (++stage == STAGES) { stage = 0; phase ^= 1; }
                }
                if (!ok) break;
                mma_commit(acc_full);
                acc_phase ^= 1;
            }
        }
    } else {
        // ------------------------------------------------ epilogue (warps 2..9)
        // warp w reads tensor-memory lanes 32*(w % 4)..+31; the two warps of a lane quarter split the columns
        const int quarter = warp & 3;
        const int half = (warp - 2) >> 2;
        uint32_t acc_phase = 0;
        int slot = 0; uint32_t sphase = 0;
        int buf = 0; uint32_t sums_phase = 0;                  // bit b: phase of sums_full[b]
        bool ok = true;
        [[maybe_unused]] int etr = 0;
        const uint32_t t_row = tmem_base + ((uint32_t)(quarter * 32) << 16);
        while (ok) {
            ok = mbar_wait(&sched_full[slot], sphase, abort_flag, q.status);
            if (!ok) break;
            const int g = sched_item[slot];
            __syncwarp();
            if (lane == 0) mbar_arrive(&sched_empty[slot]);
            if (++slot == SCHED) { slot = 0; sphase ^= 1; }
            if (g < 0) break;
            const int l = layer_of(q, g);
            const Params& p = q.layer[l];
            const bool x_is_z = p.d_out > p.d_in;
            const int e = g - q.group_begin[l];
            float val = 0.f;
#pragma unroll 1
            for (int pass = 0; pass < 2; ++pass) {
                // pass 0 = E1: 128 columns of G^X_11 (at 256) and G^Y_11 (at 384), 64 per warp;
                // pass 1 = E0: 256 columns of G^X_0 (at 0) and G^Y_0 (at 256), 128 per warp
                ok = mbar_wait(acc_full, acc_phase, abort_flag, q.status);
                if (!ok) break;
                if (threadIdx.x == 64) { DPCLIP_TRACE_AT(3, etr); ++etr; }
                acc_phase ^= 1;
                tc_fence_after_sync();
                const int width = pass == 0 ? 64 : 128;
                const uint32_t cx = (pass == 0 ? 256 : 0) + half * width, cy = (pass == 0 ? 384 : 256) + half * width;
                float sa = 0.f, sb = 0.f;
#pragma unroll 1
                for (int c0 = 0; c0 < width; c0 += 32) {
                    uint32_t vx[32], vy[32];
                    tmem_ld_32x32(t_row + cx + c0, vx);
                    tmem_ld_32x32(t_row + cy + c0, vy);
                    tmem_ld_wait();
#pragma unroll
                    for (int j = 0; j < 32; ++j) {
                        const float x = __uint_as_float(vx[j]), y = __uint_as_float(vy[j]);
                        sa = fmaf(x, y, sa);
                        sb += x_is_z ? x : y;                   // entries of Zb Zb^T: the bias term
                    }
                }
                tc_fence_before_sync();
                __syncwarp();
                if (lane == 0) mbar_arrive(acc_empty);
                if (threadIdx.x == 64) { DPCLIP_TRACE_AT(3, etr); ++etr; }
                // block (0,1) stands for its mirror image (1,0) too
                val += ((pass == 1 && half == 1) ? 2.f : 1.f) * (sa + (p.has_bias ? sb : 0.f));
            }
            if (!ok) break;
            val = warp_sum(val);
            // Two buffers suffice: a warp writes the sums of example k + 2 only after the accumulators of that
            // example were handed over, which needs the first warp's arrival for example k + 1, after its read here.
            if (lane == 0) { sums[buf * N_EPILOGUE_WARPS + (warp - 2)] = val; mbar_arrive(&sums_full[buf]); }
            if (warp == 2) {
                ok = mbar_wait(&sums_full[buf], (sums_phase >> buf) & 1u, abort_flag, q.status);
                if (!ok) break;
                if (lane == 0) {
                    float total = 0.f;
#pragma unroll
                    for (int w = 0; w < N_EPILOGUE_WARPS; ++w) total += sums[buf * N_EPILOGUE_WARPS + w];
                    p.sq[e] = total;
                }
            }
            sums_phase ^= 1u << buf;
            buf ^= 1;
        }
    }

    // ---------------------------------------------------- teardown
    if (*abort_flag) {                                      // let copies in flight land before the CTA exits
        for (int i = 0; i < 64; ++i) __nanosleep(1000);
    }
    tc_fence_before_sync();
    __syncthreads();
    if (warp == 1) { tc_fence_after_sync(); tmem_dealloc(tmem_base, 512); }
    factors_tail(q.tail);
}

// ===========================================================================
// Zb^T diag(f) A kernel (GRAD and NORM modes)
// ===========================================================================
namespace zta {
constexpr int BN = 256;                        // d_in tile  (UMMA N)
constexpr int N_TRANSFORM_WARPS = 8, N_EPILOGUE_WARPS = 8;
constexpr int THREADS = 64 + 32 * (N_TRANSFORM_WARPS + N_EPILOGUE_WARPS);   // warp 0 TMA, warp 1 MMA
constexpr int OUT_STAGE_BYTES = N_EPILOGUE_WARPS * 4096;          // 32 rows x 32 fp32 per epilogue warp
constexpr int SMEM_BYTES = 192 * 1024 + 256 + OUT_STAGE_BYTES + 1024;

// MT = number of 128-row sub-tiles of d_out per CTA tile.
//   MT = 1: 128 x 256 tile, two accumulator buffers in tensor memory (the epilogue of one item
//           overlaps the main loop of the next), 4 stages of 48 KB.
//   MT = 2: 256 x 256 tile, one accumulator buffer (all 512 columns), 3 stages of 64 KB; a third
//           less L2->SM traffic per flop, for layers where that traffic is the limit.
// Stages are 64 rows: with 32-row stages (twice as many slots) the large tile ran 10-15 % slower, the
// per-stage cost of the transform warps (barrier round trips, proxy fence) weighing twice.
template <int MT> struct Cfg {
    static constexpr int BM = 128 * MT;
    static constexpr int BK = 64;                                 // rows per stage
    static constexpr int CHUNK_BYTES = BK * 128;                  // one TMA box: BK rows x 64 bf16 columns
    static constexpr int A_BYTES = (BM / 64) * CHUNK_BYTES;       // Zb tile
    static constexpr int B_BYTES = (BN / 64) * CHUNK_BYTES;       // A tile
    static constexpr int STAGE_BYTES = A_BYTES + B_BYTES;
    static constexpr int STAGES = (192 * 1024) / STAGE_BYTES;
    static constexpr int NBUF = MT == 1 ? 2 : 1;
};

struct Params {
    int R, T, d_in, d_out;
    int norm_mode;                 // 0 = GRAD, 1 = NORM
    int tiles_m, tiles_n;          // tiles_m counts the d_out tiles of ALL layers of the launch (layer-major)
    int tiles_m_layer;             // d_out tiles of one layer (= tiles_m for a single layer)
    int n_items;
    int kb_per_split;              // GRAD: stages (blocks of Cfg::BK rows) per item
    int do_bias;                   // GRAD: gb != NULL; NORM: has_bias
    const float* clip;             // GRAD: [B] or NULL
    float* gW; long ldg; float* gb; int vec_ok;
    float* part;                   // GRAD with split rows: [n_items][BM][BN] fp32 partial tiles (workspace)
    float* bias_part;              // GRAD with split rows and a bias: [n_items][BM] partial column sums
    float* sq;                     // NORM
    int* status;
};

// Several layers of ONE shape (same R, T, d_in, d_out: e.g. the four attention projections) can share a
// GRAD launch: their d_out tiles are stacked, every item knows its layer and takes that layer's tensor
// maps, and the partial tiles of all layers go to one scratch area.  A layer of this size alone gives each
// CTA 14 stages, a third of which is pipeline fill and epilogue; four of them give 57.
constexpr int MAX_LAYERS = 8;
struct Maps { CUtensorMap a[MAX_LAYERS], z[MAX_LAYERS]; };

struct Item { int m0, n0, tn; int row_begin, row_end; int nkb; int example; int layer; };

template <int MT>
__device__ __forceinline__ Item decode(const Params& p, int item) {
    Item w;
    const int n_tiles = p.tiles_m * p.tiles_n;
    const int tile = item % n_tiles, outer = item / n_tiles;
    const int tm = tile / p.tiles_n;
    w.layer = tm / p.tiles_m_layer;
    w.m0 = (tm - w.layer * p.tiles_m_layer) * Cfg<MT>::BM;
    w.tn = tile % p.tiles_n;
    w.n0 = w.tn * BN;
    if (p.norm_mode) {
        w.example = outer;
        w.row_begin = outer * p.T;
        w.row_end = w.row_begin + p.T;
    } else {
        w.example = -1;
        w.row_begin = outer * p.kb_per_split * Cfg<MT>::BK;
        w.row_end = min(w.row_begin + p.kb_per_split * Cfg<MT>::BK, p.R);
    }
    w.nkb = (w.row_end - w.row_begin + Cfg<MT>::BK - 1) / Cfg<MT>::BK;
    return w;
}
}  // namespace zta

template <int MT>
__global__ void __launch_bounds__(zta::THREADS, 1)
zta_tc_kernel(const __grid_constant__ zta::Maps maps, const zta::Params p) {
    using namespace zta;
    using C = Cfg<MT>;
    constexpr int STAGES = C::STAGES, STAGE_BYTES = C::STAGE_BYTES, A_BYTES = C::A_BYTES, NBUF = C::NBUF;
    constexpr int BK = C::BK, CHUNK_BYTES = C::CHUNK_BYTES;
    extern __shared__ uint8_t smem_raw[];
    uint8_t* smem = smem_raw + ((1024u - (smem_u32(smem_raw) & 1023u)) & 1023u);   // 1024-byte aligned; an offset from the array keeps the accesses in the shared state space
    uint64_t* full = reinterpret_cast<uint64_t*>(smem + STAGES * STAGE_BYTES);   // TMA landed
    uint64_t* ready = full + STAGES;                                             // transform done
    uint64_t* empty = ready + STAGES;                                            // MMA done with the stage
    uint64_t* acc_full = empty + STAGES;
    uint64_t* acc_empty = acc_full + 2;
    uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(acc_empty + 2);
    volatile int* abort_flag = reinterpret_cast<volatile int*>(tmem_slot + 1);
    float4* out_stage = reinterpret_cast<float4*>(smem + STAGES * STAGE_BYTES + 256);

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    if (threadIdx.x == 0) {
        for (int s = 0; s < STAGES; ++s) {
            mbar_init(&full[s], 1); mbar_init(&ready[s], N_TRANSFORM_WARPS); mbar_init(&empty[s], 1);
        }
        for (int b = 0; b < 2; ++b) { mbar_init(&acc_full[b], 1); mbar_init(&acc_empty[b], N_EPILOGUE_WARPS); }
        *abort_flag = 0;
        mbar_fence_init();
        const int n_layers = p.tiles_m / p.tiles_m_layer;
        for (int l = 0; l < n_layers; ++l) { tma_prefetch_desc(&maps.a[l]); tma_prefetch_desc(&maps.z[l]); }
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
            int tr = 0;
            DPCLIP_TRACE_AT(0, 255);
            for (int item = blockIdx.x; item < p.n_items && ok; item += gridDim.x) {
                const Item w = decode<MT>(p, item);
                const CUtensorMap* map_a = &maps.a[w.layer];
                const CUtensorMap* map_z = &maps.z[w.layer];
                for (int kb = 0; kb < w.nkb; ++kb) {
                    ok = mbar_wait(&empty[stage], phase ^ 1, abort_flag, p.status);
                    if (!ok) break;
                    DPCLIP_TRACE_AT(0, tr); ++tr;
                    uint8_t* dst = smem + stage * STAGE_BYTES;
                    const int y = w.row_begin + kb * BK;
                    mbar_arrive_expect_tx(&full[stage], STAGE_BYTES);
#pragma unroll
                    for (int c = 0; c < C::BM / 64; ++c)
                        tma_load_2d(dst + c * CHUNK_BYTES, map_z, &full[stage], w.m0 + c * 64, y);
#pragma unroll
                    for (int c = 0; c < BN / 64; ++c)
                        tma_load_2d(dst + A_BYTES + c * CHUNK_BYTES, map_a, &full[stage], w.n0 + c * 64, y);
                    if (++stage == STAGES) { stage = 0; phase ^= 1; }
                }
            }
        }
    } else if (warp == 1) {
        // ------------------------------------------------ MMA issuer
        if (lane == 0) {
            constexpr uint32_t idesc = make_idesc_bf16(128, BN, 1, 1);
            int stage = 0; uint32_t phase = 0; int it = 0;
            bool ok = true;
            int tr = 0;
            for (int item = blockIdx.x; item < p.n_items && ok; item += gridDim.x) {
                const Item w = decode<MT>(p, item);
                const int buf = it % NBUF; const uint32_t acc_phase = (it / NBUF) & 1;
                ok = mbar_wait(&acc_empty[buf], acc_phase ^ 1, abort_flag, p.status);
                if (!ok) break;
                tc_fence_after_sync();
                for (int kb = 0; kb < w.nkb; ++kb) {
                    ok = mbar_wait(&ready[stage], phase, abort_flag, p.status);
                    if (!ok) break;
                    DPCLIP_TRACE_AT(2, tr); ++tr;
                    tc_fence_after_sync();
                    const uint32_t a_addr = smem_u32(smem + stage * STAGE_BYTES);
                    const uint32_t b_addr = a_addr + A_BYTES;
#pragma unroll
                    for (int k4 = 0; k4 < BK / 16; ++k4) {
                        // MN-major, 128-byte swizzle: 64-column chunks CHUNK_BYTES apart (leading offset),
                        // 8-row groups 1024 bytes apart (stride offset); 16 rows = 2048 bytes
                        const uint64_t db = make_smem_desc_sw128(b_addr + k4 * 2048, CHUNK_BYTES, 1024);
#pragma unroll
                        for (int h = 0; h < MT; ++h) {
                            const uint64_t da = make_smem_desc_sw128(a_addr + h * 2 * CHUNK_BYTES + k4 * 2048,
                                                                     CHUNK_BYTES, 1024);
                            mma_bf16_ss(tmem_base + (buf * MT + h) * BN, da, db, idesc,
                                        (kb == 0 && k4 == 0) ? 0u : 1u);
                        }
                    }
                    mma_commit(&empty[stage]);
                    if (++stage == STAGES) { stage = 0; phase ^= 1; }
                }
                if (!ok) break;
                mma_commit(&acc_full[buf]);
                ++it;
            }
        }
    } else if (warp < 2 + N_TRANSFORM_WARPS) {
        // ------------------------------------------------ transform (256 threads)
        // Within each 128-column half of the Zb tile, thread t owns the 8 columns [8q, 8q+8),
        // q = t / 16, on rows (t % 16) + 16 i.  Column chunk q sits at 16-byte slot q ^ (row & 7)
        // of its 128-byte row (the TMA swizzle), which is the same slot for all rows of a thread.
        const int t = threadIdx.x - 64;
        const int q = t >> 4, rs = t & 15;
        const int box = q >> 3, lq = q & 7;
        const uint32_t off = box * CHUNK_BYTES + rs * 128 + ((lq ^ (rs & 7)) << 4);
        int stage = 0; uint32_t phase = 0;
        bool ok = true;
        int tr = 0;
        for (int item = blockIdx.x; item < p.n_items && ok; item += gridDim.x) {
            const Item w = decode<MT>(p, item);
            // bias gradient = column sums of the scaled Zb tile; the values pass through these threads'
            // registers anyway, so the sums cost no extra shared-memory traffic
            float cs[MT][8];
#pragma unroll
            for (int h = 0; h < MT; ++h)
#pragma unroll
                for (int j = 0; j < 8; ++j) cs[h][j] = 0.f;
            for (int kb = 0; kb < w.nkb; ++kb) {
                // the factors of this stage's rows are fetched BEFORE waiting for the tile, so the
                // global-load latency overlaps the wait instead of sitting between TMA and MMA
                const int blk0 = w.row_begin + kb * BK;              // rows [blk0, blk0 + BK)
                const int e_first = blk0 / p.T;
                const int rem0 = blk0 - e_first * p.T;
                // fast path: the whole stage lies inside one example and inside the row range
                const bool uniform = (rem0 + BK <= p.T) && (blk0 + BK <= w.row_end);
                // GRAD: every n-tile of a row range sees the same Zb rows; the bias sums of stage kb are
                // taken by the n-tile with kb % tiles_n == tn (equal shares).  NORM: the sums must be
                // complete before they are squared, so n-tile 0 takes them all.
                const bool bias_here = p.do_bias && (p.norm_mode ? w.tn == 0 : (kb % p.tiles_n) == w.tn);
                constexpr int NR = BK / 16;                          // rows per thread and sub-tile
                float fr[NR];
#pragma unroll
                for (int i = 0; i < NR; ++i) {
                    const int rl = uniform ? 0 : rs + 16 * i;
                    float f = 1.f;
                    if (blk0 + rl >= w.row_end) f = 0.f;             // rows of another example / past the end
                    else if (p.clip) f = __ldg(p.clip + e_first + (rem0 + rl) / p.T);
                    fr[i] = f;
                }
                ok = mbar_wait(&full[stage], phase, abort_flag, p.status);
                if (!ok) break;
                if (t == 0) { DPCLIP_TRACE_AT(1, tr); ++tr; }
                uint8_t* zt = smem + stage * STAGE_BYTES;
                // packed bf16 scaling: f = f_hi + f_lo (two bf16); z*f_lo is tiny, so the fused
                // multiply-add z*f_hi + (z*f_lo) rounds the product once
                auto scale8 = [](uint4& v, float f) {
                    const __nv_bfloat16 fh = __float2bfloat16_rn(f);
                    const __nv_bfloat16 fl = __float2bfloat16_rn(f - __bfloat162float(fh));
                    const __nv_bfloat162 fh2 = __halves2bfloat162(fh, fh), fl2 = __halves2bfloat162(fl, fl);
                    __nv_bfloat162* z2 = reinterpret_cast<__nv_bfloat162*>(&v);
#pragma unroll
                    for (int u = 0; u < 4; ++u) z2[u] = __hfma2(z2[u], fh2, __hmul2(z2[u], fl2));
                };
                auto add8 = [](float* c, const uint4& v) {
                    const uint32_t wds[4] = {v.x, v.y, v.z, v.w};
#pragma unroll
                    for (int u = 0; u < 4; ++u) {
                        c[2 * u] += __uint_as_float(wds[u] << 16);
                        c[2 * u + 1] += __uint_as_float(wds[u] & 0xFFFF0000u);
                    }
                };
                if (uniform) {
                    // one factor for the whole stage: all loads are issued before the first store, so the
                    // stage costs one shared-memory round trip instead of one per row
                    const float f = fr[0];
                    if (f != 1.f || bias_here) {
                        uint4 v[MT][NR];
#pragma unroll
                        for (int h = 0; h < MT; ++h)
#pragma unroll
                            for (int i = 0; i < NR; ++i)
                                v[h][i] = *reinterpret_cast<const uint4*>(zt + h * 2 * CHUNK_BYTES + off + i * 2048);
                        if (f != 1.f) {
#pragma unroll
                            for (int h = 0; h < MT; ++h)
#pragma unroll
                                for (int i = 0; i < NR; ++i) {
                                    scale8(v[h][i], f);
                                    *reinterpret_cast<uint4*>(zt + h * 2 * CHUNK_BYTES + off + i * 2048) = v[h][i];
                                }
                        }
                        if (bias_here) {
#pragma unroll
                            for (int h = 0; h < MT; ++h)
#pragma unroll
                                for (int i = 0; i < NR; ++i) add8(cs[h], v[h][i]);
                        }
                    }
                } else {
                    // a factor per row (short examples, the ends of a row range): the same order -- all loads,
                    // then the rows that need it rewritten -- at the price of loading rows whose factor is 1
                    bool any = bias_here;
#pragma unroll
                    for (int i = 0; i < NR; ++i) any = any || fr[i] != 1.f;
                    if (any) {
                        uint4 v[MT][NR];
#pragma unroll
                        for (int h = 0; h < MT; ++h)
#pragma unroll
                            for (int i = 0; i < NR; ++i)
                                v[h][i] = *reinterpret_cast<const uint4*>(zt + h * 2 * CHUNK_BYTES + off + i * 2048);
#pragma unroll
                        for (int i = 0; i < NR; ++i) {
                            if (fr[i] != 1.f) {
#pragma unroll
                                for (int h = 0; h < MT; ++h) {
                                    scale8(v[h][i], fr[i]);
                                    *reinterpret_cast<uint4*>(zt + h * 2 * CHUNK_BYTES + off + i * 2048) = v[h][i];
                                }
                            }
                        }
                        if (bias_here) {
#pragma unroll
                            for (int h = 0; h < MT; ++h)
#pragma unroll
                                for (int i = 0; i < NR; ++i) add8(cs[h], v[h][i]);
                        }
                    }
                }
                fence_proxy_async_smem();
                __syncwarp();
                if (lane == 0) mbar_arrive(&ready[stage]);
                if (t == 0) { DPCLIP_TRACE_AT(1, tr); ++tr; }
                if (++stage == STAGES) { stage = 0; phase ^= 1; }
            }
            if (!ok) break;
            if (p.do_bias && !(p.norm_mode && w.tn != 0)) {
                // finish the column sums over the 16 row-subsets (16 consecutive lanes)
                float ssq = 0.f;
#pragma unroll
                for (int h = 0; h < MT; ++h)
#pragma unroll
                    for (int j = 0; j < 8; ++j) {
                        float c = cs[h][j];
                        c += __shfl_xor_sync(0xFFFFFFFFu, c, 1);
                        c += __shfl_xor_sync(0xFFFFFFFFu, c, 2);
                        c += __shfl_xor_sync(0xFFFFFFFFu, c, 4);
                        c += __shfl_xor_sync(0xFFFFFFFFu, c, 8);
                        ssq = fmaf(c, c, ssq);
                        if (!p.norm_mode && rs == 0) {
                            const int ml = h * 128 + q * 8 + j;
                            if (p.bias_part) p.bias_part[(size_t)item * C::BM + ml] = c;
                            else if (w.m0 + ml < p.d_out) red_add_f32(p.gb + w.m0 + ml, c);
                        }
                    }
                if (p.norm_mode) {
                    if (rs != 0) ssq = 0.f;
                    ssq = warp_sum(ssq);
                    if (lane == 0) atomicAdd(p.sq + w.example, ssq);
                }
            }
        }
    } else {
        // ------------------------------------------------ epilogue (8 warps)
        // Warp w may touch tensor-memory lanes 32*(w % 4) .. +31.  Two warps share each lane
        // quarter: group g = 0/1 takes the two column halves (MT = 1) or the two row halves (MT = 2).
        const int quarter = warp & 3;
        const int g = (warp - (2 + N_TRANSFORM_WARPS)) >> 2;
        const int ew = warp - (2 + N_TRANSFORM_WARPS);
        const int h = MT == 2 ? g : 0;
        const int col_begin = MT == 2 ? 0 : g * (BN / 2);
        const int col_end = MT == 2 ? BN : col_begin + BN / 2;
        int it = 0;
        for (int item = blockIdx.x; item < p.n_items; item += gridDim.x) {
            const Item w = decode<MT>(p, item);
            const int buf = it % NBUF; const uint32_t acc_phase = (it / NBUF) & 1;
            if (!mbar_wait(&acc_full[buf], acc_phase, abort_flag, p.status)) break;
            if (threadIdx.x == 64 + 32 * N_TRANSFORM_WARPS) DPCLIP_TRACE_AT(3, 2 * it);
            tc_fence_after_sync();
            const uint32_t t_row = tmem_base + ((uint32_t)(quarter * 32) << 16) + (buf * MT + h) * BN;
            const int m_base = w.m0 + h * 128 + quarter * 32;     // first output row of this warp
            float fro = 0.f;
#pragma unroll 1
            for (int c0 = col_begin; c0 < col_end; c0 += 32) {
                uint32_t v[32];
                tmem_ld_32x32(t_row + c0, v);
                tmem_ld_wait();
                if (p.norm_mode) {
                    // rows/columns beyond d_out/d_in were zero-filled by TMA and add nothing
#pragma unroll
                    for (int j = 0; j < 32; ++j) { const float x = __uint_as_float(v[j]); fro = fmaf(x, x, fro); }
                } else {
                    // Transpose the 32 x 32 block through shared memory so that every store/red
                    // instruction covers 4 rows x 128 contiguous bytes instead of 32 rows x 16 bytes.
                    float4* st = out_stage + ew * 256;
#pragma unroll
                    for (int j = 0; j < 8; ++j)
                        st[lane * 8 + (j ^ (lane & 7))] =
                            make_float4(__uint_as_float(v[4 * j]), __uint_as_float(v[4 * j + 1]),
                                        __uint_as_float(v[4 * j + 2]), __uint_as_float(v[4 * j + 3]));
                    __syncwarp();
                    const int jj = lane & 7;
                    const int n = w.n0 + c0 + 4 * jj;
#pragma unroll
                    for (int i = 0; i < 8; ++i) {
                        const int rr = 4 * i + (lane >> 3);
                        const float4 x = st[rr * 8 + (jj ^ (rr & 7))];
                        if (p.part) {
                            // rows split over several items: store the partial tile (dense, no bounds);
                            // reduce_partials_kernel adds the items of a tile in a fixed order
                            float* dst = p.part + ((size_t)item * C::BM + (h * 128 + quarter * 32 + rr)) * BN + c0 + 4 * jj;
                            *reinterpret_cast<float4*>(dst) = x;
                        } else {
                            const int mm = m_base + rr;
                            if (mm < p.d_out) {
                                float* dst = p.gW + (size_t)mm * p.ldg + n;
                                if (p.vec_ok && n + 4 <= p.d_in) {
                                    *reinterpret_cast<float4*>(dst) = x;
                                } else {
                                    const float xs[4] = {x.x, x.y, x.z, x.w};
#pragma unroll
                                    for (int u = 0; u < 4; ++u)
                                        if (n + u < p.d_in) dst[u] = xs[u];
                                }
                            }
                        }
                    }
                    __syncwarp();
                }
            }
            tc_fence_before_sync();
            __syncwarp();
            if (lane == 0) mbar_arrive(&acc_empty[buf]);
            if (threadIdx.x == 64 + 32 * N_TRANSFORM_WARPS) DPCLIP_TRACE_AT(3, 2 * it + 1);
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

// ---------------------------------------------------------------------------
// Second stage of the split-row clipped sum: adds the partial tiles of every
// output tile in a fixed order (deterministic, no atomics) and writes gW / gb.
// When noise_scale > 0 the Gaussian noise of element j = m*d_in + n is added in
// the same pass (requires dense rows and d_in % 4 == 0, so that a float4 of the
// output is exactly one Philox block).
// ---------------------------------------------------------------------------
struct ReduceParams {
    const float* part; const float* bias_part;
    int n_tiles, tiles_n, ksplit, BM, BN;                       // partial tiles are BM x BN fp32
    int d_out, d_in;
    float* gW; long ldg; float* gb; int vec_ok;
    int lanes;                                                  // thread rows of a CTA sharing the row slices (1..8)
    float noise_scale; uint32_t k0, k1, sw0, sw1, sb0, sb1;     // Philox key, weight / bias stream words
    // Layers of one shape that shared a GRAD launch: blockIdx.y = layer; layer y's tiles start at tile
    // y * tiles_layer of every row slice, and its outputs and noise streams come from the arrays (n_layers
    // == 0: a single layer described by the scalar fields above).
    int n_layers, tiles_layer;
    int bias_col;                                               // 1: the bias sums are column d_in of the tiles (no bias_part)
    float* gW_l[zta::MAX_LAYERS]; float* gb_l[zta::MAX_LAYERS];
    uint32_t sw0_l[zta::MAX_LAYERS], sw1_l[zta::MAX_LAYERS], sb0_l[zta::MAX_LAYERS], sb1_l[zta::MAX_LAYERS];
};

}  // namespace tc
}  // namespace dpclip

#include "kernels_stream.cuh"

namespace dpclip {
namespace tc {

__global__ void __launch_bounds__(256)
reduce_partials_kernel(const ReduceParams q) {
    __shared__ float4 part_s[256];
    ReduceParams p = q;
    if (q.n_layers > 0) {
        const int y = blockIdx.y;
        p.part = q.part + (size_t)y * q.tiles_layer * q.BM * q.BN;
        if (q.bias_part) p.bias_part = q.bias_part + (size_t)y * q.tiles_layer * q.BM;
        p.gW = q.gW_l[y]; p.gb = q.gb_l[y];
        p.sw0 = q.sw0_l[y]; p.sw1 = q.sw1_l[y]; p.sb0 = q.sb0_l[y]; p.sb1 = q.sb1_l[y];
    }
    const int n4 = (p.d_in + 3) >> 2;
    const long total = (long)p.d_out * n4;
    const size_t tile_elems = (size_t)p.BM * p.BN;
    const size_t ks_stride = (size_t)p.n_tiles * tile_elems;
    // The 256 threads of a CTA form `groups` rows of 256 / groups threads: a row covers consecutive
    // output float4s (coalesced loads) and takes every groups-th row slice; the rows' sums are then
    // combined through shared memory in a fixed order.  Small outputs with many slices get many groups,
    // so the kernel always has enough loads in flight, and the result is reproducible.
    const int groups = p.lanes, width = 256 / groups;
    const int gy = threadIdx.x / width, gx = threadIdx.x - gy * width;
    for (long idx0 = (long)blockIdx.x * width; idx0 < total; idx0 += (long)gridDim.x * width) {
        const long idx = idx0 + gx;
        const bool live = idx < total;
        const int m = live ? (int)(idx / n4) : 0, n = live ? (int)(idx % n4) << 2 : 0;
        const int tm = m / p.BM, tn = n / p.BN;
        const float* src = p.part + (size_t)(tm * p.tiles_n + tn) * tile_elems + (size_t)(m - tm * p.BM) * p.BN +
                           (n - tn * p.BN);
        float4 acc = make_float4(0.f, 0.f, 0.f, 0.f);
        if (live) {
            int ks = gy;
            for (; ks + 3 * groups < p.ksplit; ks += 4 * groups) {  // four independent loads in flight
                float4 v[4];
#pragma unroll
                for (int u = 0; u < 4; ++u) v[u] = __ldcs(reinterpret_cast<const float4*>(src + (ks + u * groups) * ks_stride));
#pragma unroll
                for (int u = 0; u < 4; ++u) { acc.x += v[u].x; acc.y += v[u].y; acc.z += v[u].z; acc.w += v[u].w; }
            }
            for (; ks < p.ksplit; ks += groups) {
                const float4 v = __ldcs(reinterpret_cast<const float4*>(src + ks * ks_stride));
                acc.x += v.x; acc.y += v.y; acc.z += v.z; acc.w += v.w;
            }
        }
        if (groups > 1) {
            __syncthreads();
            part_s[threadIdx.x] = acc;
            __syncthreads();
            if (gy == 0)
                for (int g = 1; g < groups; ++g) {
                    const float4 v = part_s[g * width + gx];
                    acc.x += v.x; acc.y += v.y; acc.z += v.z; acc.w += v.w;
                }
        }
        if (!live || gy != 0) continue;
        if (p.noise_scale > 0.f) {
            const size_t q = ((size_t)m * p.d_in + n) >> 2;
            PhiloxBlock b = philox_block((uint32_t)q, (uint32_t)(q >> 32), p.sw0, p.sw1, p.k0, p.k1);
            float z0, z1, z2, z3;
            box_muller(b.v[0], b.v[1], z0, z1);
            box_muller(b.v[2], b.v[3], z2, z3);
            acc.x = fmaf(p.noise_scale, z0, acc.x); acc.y = fmaf(p.noise_scale, z1, acc.y);
            acc.z = fmaf(p.noise_scale, z2, acc.z); acc.w = fmaf(p.noise_scale, z3, acc.w);
        }
        float* dst = p.gW + (size_t)m * p.ldg + n;
        if (p.vec_ok && n + 4 <= p.d_in) {
            *reinterpret_cast<float4*>(dst) = acc;
        } else {
            const float xs[4] = {acc.x, acc.y, acc.z, acc.w};
            for (int u = 0; u < 4; ++u)
                if (n + u < p.d_in) dst[u] = xs[u];
        }
    }
    if (p.gb) {
        // bias: one warp per output, lanes over the (row slice, n-tile) partial sums, fixed-order combine
        const int lane = threadIdx.x & 31;
        const int n_part = p.ksplit * p.tiles_n;
        for (int m = (blockIdx.x * blockDim.x + threadIdx.x) >> 5; m < p.d_out; m += (gridDim.x * blockDim.x) >> 5) {
            const int tm = m / p.BM;
            float acc = 0.f;
            if (p.bias_col) {
                // the tiles were built from [A | 1]: the sums sit in column d_in of the tile that holds it
                const int tn = p.d_in / p.BN, cb = p.d_in - tn * p.BN;
                for (int ks = lane; ks < p.ksplit; ks += 32)
                    acc += p.part[(((size_t)ks * p.n_tiles + tm * p.tiles_n + tn) * p.BM + (m - tm * p.BM)) * p.BN + cb];
            } else {
                for (int j = lane; j < n_part; j += 32) {
                    const int ks = j / p.tiles_n, tn = j - ks * p.tiles_n;
                    acc += p.bias_part[((size_t)ks * p.n_tiles + tm * p.tiles_n + tn) * p.BM + (m - tm * p.BM)];
                }
            }
            acc = warp_sum(acc);
            if (lane != 0) continue;
            if (p.noise_scale > 0.f) {
                PhiloxBlock b = philox_block((uint32_t)(m >> 2), 0u, p.sb0, p.sb1, p.k0, p.k1);
                float z[4];
                box_muller(b.v[0], b.v[1], z[0], z[1]);
                box_muller(b.v[2], b.v[3], z[2], z[3]);
                acc = fmaf(p.noise_scale, z[m & 3], acc);
            }
            p.gb[m] = acc;
        }
    }
}

}  // namespace tc
}  // namespace dpclip
