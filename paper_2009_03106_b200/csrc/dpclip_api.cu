// C ABI of libdpclip: argument checking, method selection and kernel launches.
#include <stdint.h>
#include <string.h>

#include "common.cuh"
#include <math.h>

#include "kernels_simt.cuh"
#include "kernels_stream.cuh"
#include "kernels_tc.cuh"
#include "kernels_tc_pair.cuh"
#include "kernels_fused_t1_tf32.cuh"
#include "kernels_tf32.cuh"
#include "kernels_fused_t1.cuh"
#include "kernels_narrow.cuh"
#include "kernels_narrow_tc.cuh"
#include "kernels_conv_tc.cuh"
#include "kernels_narrow_pack.cuh"
#include "kernels_elementwise.cuh"

#include <stdio.h>
#include <stdlib.h>
#include <atomic>

using namespace dpclip;

namespace {

inline size_t elt_size(dpclip_dtype dt) { return dt == DPCLIP_F32 ? 4 : 2; }
inline bool aligned_to(const void* p, size_t a) { return (reinterpret_cast<uintptr_t>(p) % a) == 0; }
inline size_t round_up(size_t x, size_t a) { return (x + a - 1) / a * a; }
// Kernels launched by this library since it was loaded (observability only; never read by a kernel).
std::atomic<unsigned long long> g_launches{0};
constexpr int kGridCounterOffset = 64;   // workspace header: status word at 0, grid-barrier counter here
constexpr int kWorkCounterOffset = 128;  // item counter of the dynamically scheduled Gram kernel (wraps to zero by itself)
constexpr int kTailCounterOffset = 192;  // CTAs done, for the factors tail of a Gram launch (reset by the last CTA)
inline int launch_status() {
    g_launches.fetch_add(1, std::memory_order_relaxed);
    return cudaGetLastError() == cudaSuccess ? DPCLIP_OK : DPCLIP_ERR_CUDA;
}

// Path switches for tests and measurements (not configuration): a bit mask read ONCE from the DPCLIP_*
// environment variables, on the first call that asks, so that no entry point touches the environment on its
// way to a launch.  dpclip_reload_path_switches() re-reads them (the tests flip a variable, reload, and
// reload again afterwards).
enum PathSwitch : unsigned {
    SW_FORCE_SIMT = 1u << 0, SW_NO_NARROW = 1u << 1, SW_NO_NARROW_RING = 1u << 2, SW_NO_NARROW_TC = 1u << 3,
    SW_NO_NARROW_PACK = 1u << 4, SW_NARROW_PACK_BF16 = 1u << 5, SW_NO_GRAM_Q2 = 1u << 6, SW_NO_T1_TF32 = 1u << 7,
    SW_NO_FUSED_T1 = 1u << 8, SW_NO_GRAM_GROUP = 1u << 9, SW_NO_GRAD_GROUP = 1u << 10, SW_NO_CONV_TC = 1u << 11,
    SW_NO_CONV_PATCHES = 1u << 12, SW_TILE_M1 = 1u << 13, SW_TILE_M2 = 1u << 14, SW_T1_TWO_LAUNCHES = 1u << 15, SW_NO_PAIR = 1u << 16, SW_LOG = 1u << 17, SW_NO_FACTORS_TAIL = 1u << 18, SW_NO_SM_BUDGET = 1u << 19, SW_NO_OVERLAP = 1u << 20,
    SW_LOADED = 1u << 31
};
std::atomic<unsigned> g_path_switches{0};
unsigned read_path_switches() {
    static const struct { const char* name; unsigned bit; char on; } table[] = {
        {"DPCLIP_FORCE_SIMT", SW_FORCE_SIMT, '1'}, {"DPCLIP_NO_NARROW", SW_NO_NARROW, '1'},
        {"DPCLIP_NO_NARROW_RING", SW_NO_NARROW_RING, '1'}, {"DPCLIP_NO_NARROW_TC", SW_NO_NARROW_TC, '1'},
        {"DPCLIP_NO_NARROW_PACK", SW_NO_NARROW_PACK, '1'}, {"DPCLIP_NARROW_PACK_BF16", SW_NARROW_PACK_BF16, '1'},
        {"DPCLIP_NO_GRAM_Q2", SW_NO_GRAM_Q2, '1'}, {"DPCLIP_NO_T1_TF32", SW_NO_T1_TF32, '1'},
        {"DPCLIP_NO_FUSED_T1", SW_NO_FUSED_T1, '1'}, {"DPCLIP_NO_GRAM_GROUP", SW_NO_GRAM_GROUP, '1'},
        {"DPCLIP_NO_GRAD_GROUP", SW_NO_GRAD_GROUP, '1'}, {"DPCLIP_NO_CONV_TC", SW_NO_CONV_TC, '1'},
        {"DPCLIP_NO_CONV_PATCHES", SW_NO_CONV_PATCHES, '1'}, {"DPCLIP_TILE_M", SW_TILE_M1, '1'},
        {"DPCLIP_TILE_M", SW_TILE_M2, '2'}, {"DPCLIP_T1_ONE_LAUNCH", SW_T1_TWO_LAUNCHES, '0'},
        {"DPCLIP_NO_PAIR", SW_NO_PAIR, '1'}, {"DPCLIP_LOG", SW_LOG, '1'},
        {"DPCLIP_NO_FACTORS_TAIL", SW_NO_FACTORS_TAIL, '1'}, {"DPCLIP_NO_SM_BUDGET", SW_NO_SM_BUDGET, '1'},
        {"DPCLIP_NO_OVERLAP", SW_NO_OVERLAP, '1'},
    };
    unsigned v = SW_LOADED;
    for (const auto& e : table) {
        const char* env = getenv(e.name);
        if (env && env[0] == e.on) v |= e.bit;
    }
    g_path_switches.store(v, std::memory_order_relaxed);
    return v;
}
inline bool path_switch(unsigned bit) {
    unsigned v = g_path_switches.load(std::memory_order_relaxed);
    if (!(v & SW_LOADED)) v = read_path_switches();
    return (v & bit) != 0;
}

// SM budget of the calling thread's next launches (0 = the whole GPU).  A step that spreads small layers over
// several streams gives each launch a share of the SMs in proportion to its bytes: launches of a few
// megabytes are chains of round trips, not throughput problems, so running four of them side by side on a
// quarter of the SMs each costs each one little and hides the others' latency; launched at full width they
// queue for the SMs (one CTA per SM) and run one after the other.
thread_local int t_sm_budget = 0;
inline int sm_budget() { return t_sm_budget > 0 && t_sm_budget < kNumSMs ? t_sm_budget : kNumSMs; }
// Set while the next clipped-sum launch of this thread directly follows, in its stream, the Gram launch whose tail
// computed the factors: the launch then asks for programmatic serialization (see griddep_wait in tc_common.cuh).
thread_local bool t_overlap_prev = false;
struct OverlapPrevScope {
    bool prev;
    explicit OverlapPrevScope(bool on) : prev(t_overlap_prev) { t_overlap_prev = on; }
    ~OverlapPrevScope() { t_overlap_prev = prev; }
};
struct SmBudgetScope {
    int prev;
    explicit SmBudgetScope(int b) : prev(t_sm_budget) { t_sm_budget = b; }
    ~SmBudgetScope() { t_sm_budget = prev; }
};

// DPCLIP_LOG=1: one line on stderr per dispatch decision (which form of a kernel a layer takes and how its
// work is cut) -- host side only, nothing changes on the device.
#define DPCLIP_LOGF(...) do { if (path_switch(SW_LOG)) { fprintf(stderr, "[dpclip] " __VA_ARGS__); fputc('\n', stderr); } } while (0)

int check_layer_args(const void* A, long lda, const void* Z, long ldz, int B, int T, int d_in, int d_out,
                     dpclip_dtype dtype) {
    if (!A || !Z) return DPCLIP_ERR_INVALID_ARG;
    if (B <= 0 || T <= 0 || d_in <= 0 || d_out <= 0) return DPCLIP_ERR_INVALID_ARG;
    if (lda < d_in || ldz < d_out) return DPCLIP_ERR_INVALID_ARG;
    if (dtype != DPCLIP_F32 && dtype != DPCLIP_BF16) return DPCLIP_ERR_INVALID_ARG;
    if ((long)B * T > 0x7FFFFFFFL) return DPCLIP_ERR_INVALID_ARG;
    if (!aligned_to(A, elt_size(dtype)) || !aligned_to(Z, elt_size(dtype))) return DPCLIP_ERR_MISALIGNED;
    return DPCLIP_OK;
}

// 4-element vector loads need the base and every row start on a 4-element boundary.
inline int vec4_ok(const void* p, long ld, dpclip_dtype dt) {
    return aligned_to(p, 4 * elt_size(dt)) && (ld % 4 == 0);
}

void fill_simt_params(SimtParams& p, const void* A, long lda, const void* Z, long ldz, int T, int d_in,
                      int d_out, int has_bias, dpclip_dtype dtype) {
    memset(&p, 0, sizeof(p));
    p.A = A; p.lda = lda; p.Z = Z; p.ldz = ldz;
    p.T = T; p.d_in = d_in; p.d_out = d_out; p.has_bias = has_bias ? 1 : 0;
    p.tiles_m = ceil_div(d_out, SIMT_BM);
    p.tiles_n = ceil_div(d_in + p.has_bias, SIMT_BN);
    p.vec_a = vec4_ok(A, lda, dtype);
    p.vec_z = vec4_ok(Z, ldz, dtype);
}

int launch_t1_norms(const void* A, long lda, const void* Z, long ldz, int B, int d_in, int d_out,
                    dpclip_dtype dtype, int has_bias, float* sq, cudaStream_t st) {
    const int va = vec4_ok(A, lda, dtype), vz = vec4_ok(Z, ldz, dtype);
    if (dtype == DPCLIP_F32)
        t1_sqnorm_kernel<float><<<B, 256, 0, st>>>((const float*)A, lda, (const float*)Z, ldz, d_in, d_out,
                                                   has_bias, va, vz, sq);
    else
        t1_sqnorm_kernel<__nv_bfloat16><<<B, 256, 0, st>>>((const __nv_bfloat16*)A, lda,
                                                           (const __nv_bfloat16*)Z, ldz, d_in, d_out,
                                                           has_bias, va, vz, sq);
    return launch_status();
}

// narrow layers (d_in + bias <= 32, d_out <= 64, T > 1): streaming kernel with one lane per column
inline bool narrow_layer(int T, int d_in, int d_out, int has_bias, long lda, long ldz) {
    if (path_switch(SW_NO_NARROW)) return false;
    // dense rows: a run of rows is then one contiguous run of memory, which is what the kernel streams
    return T > 1 && d_in + (has_bias ? 1 : 0) <= 32 && d_out <= 64 && lda == d_in && ldz == d_out;
}

template <typename T, int MAXM, bool GRAD>
int launch_narrow_inst(const NarrowParams& p, int grid, cudaStream_t st) {
    constexpr int smem = NarrowCfg<MAXM>::SMEM_BYTES;
    if (cudaFuncSetAttribute(narrow_kernel<T, MAXM, GRAD>, cudaFuncAttributeMaxDynamicSharedMemorySize, smem) !=
        cudaSuccess) return DPCLIP_ERR_CUDA;
    narrow_kernel<T, MAXM, GRAD><<<grid, NARROW_THREADS, smem, st>>>(p);
    return launch_status();
}

template <int MAXM, int WARPS, bool GRAD>
int launch_narrow_ring_inst(const NarrowParams& p, int grid, cudaStream_t st) {
    constexpr int smem = NarrowRingCfg<MAXM, WARPS>::SMEM_BYTES;
    if (cudaFuncSetAttribute(narrow_ring_kernel<MAXM, WARPS, GRAD>, cudaFuncAttributeMaxDynamicSharedMemorySize, smem) !=
        cudaSuccess) return DPCLIP_ERR_CUDA;
    narrow_ring_kernel<MAXM, WARPS, GRAD><<<grid, 32 * WARPS, smem, st>>>(p);
    return launch_status();
}

// fp32 with every 16-row chunk starting on a 16-byte boundary (in A and in Zb): the cp.async ring form
inline bool narrow_ring_ok(const NarrowParams& p, dpclip_dtype dtype, bool grad) {
    if (path_switch(SW_NO_NARROW_RING)) return false;
    if (dtype != DPCLIP_F32 || !aligned_to(p.A, 16) || !aligned_to(p.Z, 16)) return false;
    // chunk starts are multiples of 16 rows from the slice start: 16 * d * 4 bytes is always a multiple of 16;
    // the slice start itself is a multiple of 32 rows (GRAD) or of T rows (NORM)
    if (!grad && (((long)p.T * p.d_in) % 4 != 0 || ((long)p.T * p.d_out) % 4 != 0)) return false;
    return true;
}

// bf16 narrow layers on the tensor cores: needs the status word of a workspace for its bounded waits, and
// items (examples, row slices) that start and end on 16-byte boundaries in both inputs, which the bulk copies
// into shared memory ask for
inline bool narrow_tc_ok(const NarrowParams& p, dpclip_dtype dtype, const int* status) {
    if (path_switch(SW_NO_NARROW_TC)) return false;
    if (dtype != DPCLIP_BF16 || status == nullptr) return false;
    if (!aligned_to(p.A, 16) || !aligned_to(p.Z, 16)) return false;
    return ((long)p.T * p.d_in) % 8 == 0 && ((long)p.T * p.d_out) % 8 == 0;
}

template <bool GRAD>
int launch_narrow_tc(const NarrowParams& p, int grid, int n_items, int* status, cudaStream_t st) {
    namespace n = tc::ntc;
    n::Params q;
    memset(&q, 0, sizeof(q));
    q.A = static_cast<const __nv_bfloat16*>(p.A); q.Z = static_cast<const __nv_bfloat16*>(p.Z);
    q.T = p.T; q.d_in = p.d_in; q.d_out = p.d_out; q.has_bias = p.has_bias;
    q.n_items = n_items; q.rows_total = p.rows_total; q.rows_per_cta = p.rows_per_cta;
    q.clip = p.clip; q.sq = p.sq; q.part = p.part; q.part_m = p.d_out <= 32 ? 32 : 64;
    q.status = status;
    if (!GRAD && p.d_out > 32 && cudaMemsetAsync(p.sq, 0, sizeof(float) * (size_t)n_items, st) != cudaSuccess)
        return DPCLIP_ERR_CUDA;
    if (cudaFuncSetAttribute(tc::narrow_tc_kernel<GRAD>, cudaFuncAttributeMaxDynamicSharedMemorySize, n::SMEM_BYTES) !=
        cudaSuccess) return DPCLIP_ERR_CUDA;
    tc::narrow_tc_kernel<GRAD><<<grid, n::THREADS, n::SMEM_BYTES, st>>>(q);
    return launch_status();
}

// Narrow layers with d_out <= 32 on the tensor cores, four row groups per instruction (either dtype): the same
// conditions as narrow_tc_ok, on 16-byte multiples of the element size
inline bool narrow_pack_ok(const NarrowParams& p, dpclip_dtype dtype, const int* status) {
    if (path_switch(SW_NO_NARROW_TC)) return false;
    if (path_switch(SW_NO_NARROW_PACK)) return false;
    if (status == nullptr || p.d_out > 32 || p.d_in + p.has_bias > 32) return false;
    if (dtype == DPCLIP_BF16) {
        // bf16 has few instructions to save (one per 16 rows) and pays for the extra pass through shared memory in
        // the epilogue: measured 16.4 / 18.0 us against 15.2 / 17.9 us for the unpacked kernel on the first
        // convolution of the CNN.  Kept selectable for measurements.
        if (!path_switch(SW_NARROW_PACK_BF16)) return false;
    }
    if (!aligned_to(p.A, 16) || !aligned_to(p.Z, 16)) return false;
    const long es = elt_size(dtype);
    return ((long)p.T * p.d_in * es) % 16 == 0 && ((long)p.T * p.d_out * es) % 16 == 0;
}

template <typename T, bool GRAD>
int launch_narrow_pack_inst(const tc::npk::Params& q, int grid, cudaStream_t st) {
    using Cfg = tc::npk::Cfg<T>;
    if (cudaFuncSetAttribute(tc::narrow_pack_kernel<T, GRAD>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                             Cfg::SMEM_BYTES) != cudaSuccess) return DPCLIP_ERR_CUDA;
    tc::narrow_pack_kernel<T, GRAD><<<grid, tc::npk::THREADS, Cfg::SMEM_BYTES, st>>>(q);
    return launch_status();
}

template <bool GRAD>
int launch_narrow_pack(const NarrowParams& p, int grid, int n_items, dpclip_dtype dtype, int* status, cudaStream_t st) {
    tc::npk::Params q;
    memset(&q, 0, sizeof(q));
    q.A = p.A; q.Z = p.Z; q.T = p.T; q.d_in = p.d_in; q.d_out = p.d_out; q.has_bias = p.has_bias;
    q.n_items = n_items; q.rows_total = p.rows_total; q.rows_per_cta = p.rows_per_cta;
    q.clip = p.clip; q.sq = p.sq; q.part = p.part; q.status = status;
    if (!GRAD && cudaMemsetAsync(p.sq, 0, sizeof(float) * (size_t)n_items, st) != cudaSuccess) return DPCLIP_ERR_CUDA;
    return dtype == DPCLIP_F32 ? launch_narrow_pack_inst<float, GRAD>(q, grid, st)
                               : launch_narrow_pack_inst<__nv_bfloat16, GRAD>(q, grid, st);
}

template <bool GRAD>
int launch_narrow(const NarrowParams& p, int grid, int d_out, dpclip_dtype dtype, cudaStream_t st) {
    if (narrow_ring_ok(p, dtype, GRAD)) {
        // two 8-warp CTAs per SM when there are CTAs enough for that, else one 16-warp CTA
        if (grid > kNumSMs)
            return d_out <= 32 ? launch_narrow_ring_inst<32, 8, GRAD>(p, grid, st) : launch_narrow_ring_inst<64, 8, GRAD>(p, grid, st);
        return d_out <= 32 ? launch_narrow_ring_inst<32, 16, GRAD>(p, grid, st) : launch_narrow_ring_inst<64, 16, GRAD>(p, grid, st);
    }
    if (dtype == DPCLIP_F32)
        return d_out <= 32 ? launch_narrow_inst<float, 32, GRAD>(p, grid, st) : launch_narrow_inst<float, 64, GRAD>(p, grid, st);
    return d_out <= 32 ? launch_narrow_inst<__nv_bfloat16, 32, GRAD>(p, grid, st)
                       : launch_narrow_inst<__nv_bfloat16, 64, GRAD>(p, grid, st);
}

int launch_simt_norms(const void* A, long lda, const void* Z, long ldz, int B, int T, int d_in, int d_out,
                      dpclip_dtype dtype, int has_bias, float* sq, cudaStream_t st, int* status = nullptr) {
    if (narrow_layer(T, d_in, d_out, has_bias, lda, ldz)) {
        NarrowParams q;
        memset(&q, 0, sizeof(q));
        q.A = A; q.lda = lda; q.Z = Z; q.ldz = ldz; q.T = T; q.d_in = d_in; q.d_out = d_out;
        q.has_bias = has_bias ? 1 : 0; q.sq = sq;
        if (narrow_pack_ok(q, dtype, status))
            return launch_narrow_pack<false>(q, B < sm_budget() ? B : sm_budget(), B, dtype, status, st);
        if (narrow_tc_ok(q, dtype, status))
            return launch_narrow_tc<false>(q, B < sm_budget() ? B : sm_budget(), B, status, st);
        return launch_narrow<false>(q, B, d_out, dtype, st);
    }
    SimtParams p;
    fill_simt_params(p, A, lda, Z, ldz, T, d_in, d_out, has_bias, dtype);
    const int n_tiles = p.tiles_m * p.tiles_n;
    int split = ceil_div(2 * kNumSMs, B);
    if (split > n_tiles) split = n_tiles;
    if (split < 1) split = 1;
    p.sq = sq;
    p.use_atomic = split > 1;
    if (p.use_atomic && cudaMemsetAsync(sq, 0, sizeof(float) * (size_t)B, st) != cudaSuccess)
        return DPCLIP_ERR_CUDA;
    dim3 grid(split, B);
    if (dtype == DPCLIP_F32) zta_simt_kernel<float, false><<<grid, SIMT_THREADS, 0, st>>>(p);
    else zta_simt_kernel<__nv_bfloat16, false><<<grid, SIMT_THREADS, 0, st>>>(p);
    return launch_status();
}

struct NoiseSpec { float scale; unsigned long long seed, sid_w, sid_b; };

int launch_simt_grad(const void* A, long lda, const void* Z, long ldz, int B, int T, int d_in, int d_out,
                     dpclip_dtype dtype, const float* clip, float* gW, long ldg, float* gb, cudaStream_t st,
                     void* workspace = nullptr, size_t workspace_bytes = 0, const NoiseSpec* noise = nullptr,
                     bool* noise_done = nullptr) {
    if (narrow_layer(T, d_in, d_out, gb != nullptr, lda, ldz)) {
        NarrowParams q;
        memset(&q, 0, sizeof(q));
        q.A = A; q.lda = lda; q.Z = Z; q.ldz = ldz; q.T = T; q.d_in = d_in; q.d_out = d_out;
        q.has_bias = gb ? 1 : 0; q.clip = clip; q.gW = gW; q.ldg = ldg; q.gb = gb;
        q.rows_total = (long)B * T;
        int* status = (workspace && workspace_bytes >= (size_t)kHeaderBytes) ? static_cast<int*>(workspace) : nullptr;
        const bool on_pack = narrow_pack_ok(q, dtype, status);
        const bool on_tc = on_pack || narrow_tc_ok(q, dtype, status);
        // one wave: a CTA of the register-staged kernel holds a whole SM; the cp.async form runs two per SM
        int grid = (!on_tc && narrow_ring_ok(q, dtype, true)) ? 2 * sm_budget() : sm_budget();
        const long min_rows = NARROW_WARPS * 32;                   // at least one chunk per warp
        if ((long)grid * min_rows > q.rows_total) grid = (int)((q.rows_total + min_rows - 1) / min_rows);
        // whole 32-row chunks per CTA: every chunk of a dense layer then starts on a 16-byte boundary whatever
        // the row length, and takes the 128-bit load path (a slice starting mid-chunk falls back to scalar loads)
        q.rows_per_cta = ((q.rows_total + grid - 1) / grid + 31) / 32 * 32;
        grid = (int)((q.rows_total + q.rows_per_cta - 1) / q.rows_per_cta);
        const int maxm = d_out <= 32 ? 32 : 64;
        const int parts_per_cta = 1;
        const size_t part_bytes = (size_t)grid * parts_per_cta * maxm * 32 * 4;
        if (workspace && workspace_bytes >= (size_t)kHeaderBytes + part_bytes && grid > 1) {
            // partial tile per CTA, then a fixed-order reduce that also adds the noise
            q.part = reinterpret_cast<float*>(static_cast<char*>(workspace) + kHeaderBytes);
            int rc = on_pack ? launch_narrow_pack<true>(q, grid, 1, dtype, status, st)
                   : on_tc   ? launch_narrow_tc<true>(q, grid, 1, status, st)
                             : launch_narrow<true>(q, grid, d_out, dtype, st);
            if (rc) return rc;
            NarrowReduceParams r;
            memset(&r, 0, sizeof(r));
            r.part = q.part; r.n_parts = grid * parts_per_cta; r.maxm = maxm; r.d_out = d_out; r.d_in = d_in; r.has_bias = gb ? 1 : 0;
            r.gW = gW; r.ldg = ldg; r.gb = gb;
            if (noise && noise->scale > 0.f && ldg == d_in) {
                r.noise_scale = noise->scale;
                r.k0 = (uint32_t)noise->seed; r.k1 = (uint32_t)(noise->seed >> 32);
                r.sid_w = noise->sid_w; r.sid_b = noise->sid_b;
                if (noise_done) *noise_done = true;
            }
            narrow_reduce_kernel<<<d_out, 256, 0, st>>>(r);
            return launch_status();
        }
        if (cudaMemset2DAsync(gW, sizeof(float) * (size_t)ldg, 0, sizeof(float) * (size_t)d_in, d_out, st) !=
            cudaSuccess) return DPCLIP_ERR_CUDA;
        if (gb && cudaMemsetAsync(gb, 0, sizeof(float) * (size_t)d_out, st) != cudaSuccess) return DPCLIP_ERR_CUDA;
        return launch_narrow<true>(q, grid, d_out, dtype, st);
    }
    SimtParams p;
    fill_simt_params(p, A, lda, Z, ldz, T, d_in, d_out, gb != nullptr, dtype);
    const int n_tiles = p.tiles_m * p.tiles_n;
    const long rows = (long)B * T;
    long ksplit = ceil_div(4 * kNumSMs, n_tiles);
    const long max_split = (rows + 4 * SIMT_BK - 1) / (4 * SIMT_BK);     // at least 64 rows per slice
    if (ksplit > max_split) ksplit = max_split;
    if (ksplit < 1) ksplit = 1;
    if (ksplit > 65535) ksplit = 65535;
    long per = (rows + ksplit - 1) / ksplit;
    per = (per + SIMT_BK - 1) / SIMT_BK * SIMT_BK;
    ksplit = (rows + per - 1) / per;
    p.clip = clip; p.gW = gW; p.ldg = ldg; p.gb = gb;
    p.rows_total = rows; p.rows_per_split = per;
    p.use_atomic = ksplit > 1;
    if (p.use_atomic) {
        if (cudaMemset2DAsync(gW, sizeof(float) * (size_t)ldg, 0, sizeof(float) * (size_t)d_in, d_out, st) !=
            cudaSuccess) return DPCLIP_ERR_CUDA;
        if (gb && cudaMemsetAsync(gb, 0, sizeof(float) * (size_t)d_out, st) != cudaSuccess)
            return DPCLIP_ERR_CUDA;
    }
    dim3 grid(n_tiles, (unsigned)ksplit);
    if (dtype == DPCLIP_F32) zta_simt_kernel<float, true><<<grid, SIMT_THREADS, 0, st>>>(p);
    else zta_simt_kernel<__nv_bfloat16, true><<<grid, SIMT_THREADS, 0, st>>>(p);
    return launch_status();
}


// ---------------------------------------------------------------------------
// tensor-core paths (bf16): tensor maps + launches
// ---------------------------------------------------------------------------
typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*,
                                  const cuuint64_t*, const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave,
                                  CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

EncodeTiledFn encode_tiled_fn() {
    static EncodeTiledFn fn = nullptr;       // a driver entry point, looked up once; not device state
    if (!fn) {
        void* ptr = nullptr;
        cudaDriverEntryPointQueryResult qres;
        if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &ptr, cudaEnableDefault, &qres) == cudaSuccess &&
            qres == cudaDriverEntryPointSuccess)
            fn = reinterpret_cast<EncodeTiledFn>(ptr);
    }
    return fn;
}

// 2-D bf16 matrix [rows][cols] with row stride ld elements; box = box_cols x box_rows, 128-byte swizzle,
// out-of-range elements read as zero.
bool make_map_bf16(CUtensorMap* map, const void* base, long rows, long cols, long ld, int box_cols, int box_rows,
                   bool swizzle = true) {
    EncodeTiledFn fn = encode_tiled_fn();
    if (!fn) return false;
    cuuint64_t dims[2] = {(cuuint64_t)cols, (cuuint64_t)rows};
    cuuint64_t strides[1] = {(cuuint64_t)ld * 2};
    cuuint32_t box[2] = {(cuuint32_t)box_cols, (cuuint32_t)box_rows};
    cuuint32_t estr[2] = {1, 1};
    return fn(map, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, const_cast<void*>(base), dims, strides, box, estr,
              CU_TENSOR_MAP_INTERLEAVE_NONE, swizzle ? CU_TENSOR_MAP_SWIZZLE_128B : CU_TENSOR_MAP_SWIZZLE_NONE,
              CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
              CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

// TMA needs 16-byte aligned bases and row strides.
inline bool tc_eligible(const void* A, long lda, const void* Z, long ldz, dpclip_dtype dtype) {
    if (dtype != DPCLIP_BF16) return false;
    if (path_switch(SW_FORCE_SIMT)) return false;
    return aligned_to(A, 16) && aligned_to(Z, 16) && lda % 8 == 0 && ldz % 8 == 0;
}

template <typename K>
bool enable_smem(K kernel, int bytes) {
    return cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, bytes) == cudaSuccess;
}

// One layer of a Gram-norm launch.
struct GramLayer {
    const void* A; long lda; const void* Z; long ldz;
    int B, T, d_in, d_out, has_bias;
    float* sq;
};

// every item is on the diagonal when an example spans at most two aligned row blocks
inline bool gram_diag_only(int T) {
    namespace g = tc::gram;
    return (T % g::BM == 0 && T <= 2 * g::BM) || (g::BM % T == 0);
}

// Which Gram kernel a layer takes; layers of one class can share a launch.
//   0: examples of exactly two row blocks (their own kernel: one HBM pass per example)
//   1: other layers whose items all sit on the diagonal (stages of two tiles, six of them)
//   2: the rest
inline int gram_class(int T) {
    if (path_switch(SW_NO_GRAM_Q2)) return gram_diag_only(T) ? 1 : 2;
    if (T == 2 * tc::gram::BM) return 0;
    return gram_diag_only(T) ? 1 : 2;
}

// Norms of up to gram::MAX_LAYERS layers by the Gram identity in ONE launch.  All layers must agree on
// gram_class(T).  Layers go in descending order of bytes per group, so that the round-robin deal
// leaves the small items for the end of every CTA's queue.
int launch_gram_group(const GramLayer* ls, int n, int* status, cudaStream_t st,
                      const tc::gram::FactorsTail* tail = nullptr) {
    namespace g = tc::gram;
    if (n <= 0 || n > g::MAX_LAYERS) return DPCLIP_ERR_INVALID_ARG;
    int order[g::MAX_LAYERS];
    for (int i = 0; i < n; ++i) order[i] = i;
    auto cost = [&](int i) {
        const long rows = ls[i].T % g::BM == 0 ? ls[i].T : g::BM;
        return rows * (long)(ls[i].d_in + ls[i].d_out);
    };
    for (int i = 1; i < n; ++i)                       // insertion sort, stable
        for (int j = i; j > 0 && cost(order[j]) > cost(order[j - 1]); --j) { const int t = order[j]; order[j] = order[j - 1]; order[j - 1] = t; }
    static_assert(sizeof(g::Launch) <= 4096, "kernel parameter space");
    g::Launch q;
    memset(&q, 0, sizeof(q));
    q.L = n; q.status = status;
    const int cls = gram_class(ls[0].T);
    int groups = 0;
    for (int k = 0; k < n; ++k) {
        const GramLayer& y = ls[order[k]];
        if (gram_class(y.T) != cls) return DPCLIP_ERR_INVALID_ARG;
        const long R = (long)y.B * y.T;
        if (!make_map_bf16(&q.map_a[k], y.A, R, y.d_in, y.lda, g::BK, g::BM) ||
            !make_map_bf16(&q.map_z[k], y.Z, R, y.d_out, y.ldz, g::BK, g::BM))
            return DPCLIP_ERR_CUDA;
        g::Params& p = q.layer[k];
        p.R = (int)R; p.T = y.T; p.d_in = y.d_in; p.d_out = y.d_out; p.has_bias = y.has_bias ? 1 : 0;
        p.sq = y.sq;
        if (y.T % g::BM == 0) {
            p.dense = 1; p.q = y.T / g::BM;
            p.n_groups = y.B;                     // one example per group
        } else {
            p.dense = 0;
            p.n_groups = ceil_div(R, g::BM);      // one 128-row block per group
        }
        q.group_begin[k] = groups;
        groups += p.n_groups;
    }
    // the general kernels accumulate with atomics: clear the rows, adjacent rows of sq in one memset (the kernel
    // for examples of two row blocks stores every norm, so its rows need no clearing)
    if (cls != 0) {
        int by_ptr[g::MAX_LAYERS];
        for (int i = 0; i < n; ++i) by_ptr[i] = i;
        for (int i = 1; i < n; ++i)
            for (int j = i; j > 0 && ls[by_ptr[j]].sq < ls[by_ptr[j - 1]].sq; --j) { const int t = by_ptr[j]; by_ptr[j] = by_ptr[j - 1]; by_ptr[j - 1] = t; }
        for (int i = 0; i < n;) {
            float* begin = ls[by_ptr[i]].sq;
            float* end = begin + ls[by_ptr[i]].B;
            int j = i + 1;
            while (j < n && ls[by_ptr[j]].sq == end) { end += ls[by_ptr[j]].B; ++j; }
            if (cudaMemsetAsync(begin, 0, sizeof(float) * (size_t)(end - begin), st) != cudaSuccess) return DPCLIP_ERR_CUDA;
            i = j;
        }
    }
    q.group_begin[n] = groups;
    q.total_groups = groups;
    if (tail) {
        q.tail = *tail;
        q.tail.done = reinterpret_cast<unsigned int*>(reinterpret_cast<char*>(status) + kTailCounterOffset);
    }
    const int grid = groups < sm_budget() ? groups : sm_budget();
    if (cls == 0) {
        q.work_counter = reinterpret_cast<unsigned int*>(reinterpret_cast<char*>(status) + kWorkCounterOffset);
        if (!enable_smem(tc::gram_norm_q2_kernel, g::SMEM_BYTES)) return DPCLIP_ERR_CUDA;
        tc::gram_norm_q2_kernel<<<grid, g::THREADS, g::SMEM_BYTES, st>>>(q);
    } else if (cls == 1) {
        if (!enable_smem(tc::gram_norm_kernel<true>, g::SMEM_BYTES)) return DPCLIP_ERR_CUDA;
        tc::gram_norm_kernel<true><<<grid, g::THREADS, g::SMEM_BYTES, st>>>(q);
    } else {
        if (!enable_smem(tc::gram_norm_kernel<false>, g::SMEM_BYTES)) return DPCLIP_ERR_CUDA;
        tc::gram_norm_kernel<false><<<grid, g::THREADS, g::SMEM_BYTES, st>>>(q);
    }
    return launch_status();
}

int launch_gram_norms(const void* A, long lda, const void* Z, long ldz, int B, int T, int d_in, int d_out,
                      int has_bias, float* sq, int* status, cudaStream_t st) {
    const GramLayer y = {A, lda, Z, ldz, B, T, d_in, d_out, has_bias, sq};
    return launch_gram_group(&y, 1, status, st);
}

// Largest scratch the split-row clipped sum can ask for: one partial tile per item, at most one
// wave of 256 x 256 tiles or two waves of 128 x 256 tiles, plus the partial bias sums.
constexpr size_t kTcScratchBytes = (size_t)kNumSMs * 256 * 256 * 4 + (size_t)2 * kNumSMs * 256 * 4;

// Row split of the bf16 tensor-core clipped sum: how many row slices each output tile is cut into.
//   one wave  : floor(per_sm * SMs / tiles) slices -- every CTA one item (two for the small tile when they
//               stay long); its partial tiles fit the fixed scratch above.
//   preferred : when one wave would leave more than 5 % of the SMs idle (64 tiles of 256 x 256: 128 of 148)
//               and the row ranges stay long (>= 192 stages of 64 rows, so that pipeline fill and epilogue
//               stay below 4 % of an item), the smallest split whose items fill whole waves to >= 97 %; it
//               needs one partial tile per item, which the workspace query reports for the layer.
struct ZtaSplit { int one_wave, preferred; };
inline ZtaSplit zta_pick_split(long nkb, int tiles, int per_sm, int slots = kNumSMs) {
    ZtaSplit r;
    long base = ((long)per_sm * slots) / tiles;
    if (base > nkb) base = nkb;
    if (base < 1) base = 1;
    r.one_wave = r.preferred = (int)base;
    auto fill = [&](long ks) {
        const long items = (long)tiles * ks, waves = (items + slots - 1) / slots;
        return (double)items / (double)(waves * slots);
    };
    double best = fill(base);
    if (per_sm != 1 || best >= 0.95) return r;
    for (long ks = base + 1; ks <= 64 * base && nkb / ks >= 192; ++ks) {
        const double f = fill(ks);
        if (f > best + 0.01) { best = f; r.preferred = (int)ks; if (f >= 0.97) break; }
    }
    return r;
}
inline size_t zta_scratch_bytes(int tiles, int ksplit, int BM, bool bias) {
    return (size_t)tiles * ksplit * ((size_t)BM * 256 * 4 + (bias ? (size_t)BM * 4 : 0));
}

// second stage of a split-row clipped sum: fixed-order sum of the partial tiles (+ optional noise)
// Layers of one shape that share a clipped-sum launch (n == 0: a single layer).
struct GradGroup {
    int n;
    float* gW[tc::zta::MAX_LAYERS]; float* gb[tc::zta::MAX_LAYERS];
    unsigned long long sid_w[tc::zta::MAX_LAYERS], sid_b[tc::zta::MAX_LAYERS];
};

int launch_reduce_partials(const tc::zta::Params& p, int tiles, int ksplit, int BM, int BN, int d_in, int d_out,
                           float* gW, long ldg, float* gb, const NoiseSpec* noise, bool* noise_done,
                           cudaStream_t st, const GradGroup* grp = nullptr) {
    tc::ReduceParams r;
    memset(&r, 0, sizeof(r));
    if (grp && grp->n > 0) {
        r.n_layers = grp->n; r.tiles_layer = tiles / grp->n;
        for (int l = 0; l < grp->n; ++l) {
            r.gW_l[l] = grp->gW[l]; r.gb_l[l] = grp->gb[l];
            r.sw0_l[l] = (uint32_t)grp->sid_w[l]; r.sw1_l[l] = (uint32_t)(grp->sid_w[l] >> 32);
            r.sb0_l[l] = (uint32_t)grp->sid_b[l]; r.sb1_l[l] = (uint32_t)(grp->sid_b[l] >> 32);
        }
    }
    r.part = p.part; r.bias_part = p.bias_part;
    r.n_tiles = tiles; r.tiles_n = p.tiles_n; r.ksplit = ksplit; r.BM = BM; r.BN = BN;
    r.d_out = d_out; r.d_in = d_in; r.gW = gW; r.ldg = ldg; r.gb = gb; r.vec_ok = p.vec_ok;
    if (noise && noise->scale > 0.f && ldg == d_in && d_in % 4 == 0) {
        r.noise_scale = noise->scale;
        r.k0 = (uint32_t)noise->seed; r.k1 = (uint32_t)(noise->seed >> 32);
        r.sw0 = (uint32_t)noise->sid_w; r.sw1 = (uint32_t)(noise->sid_w >> 32);
        r.sb0 = (uint32_t)noise->sid_b; r.sb1 = (uint32_t)(noise->sid_b >> 32);
        if (noise_done) *noise_done = true;
    }
    const long n_vec = (long)d_out * ((d_in + 3) / 4);
    // split the row slices over up to 8 thread rows per CTA until the grid has about two CTAs per SM
    int lanes = 1;
    while (lanes < 8 && lanes * 2 <= ksplit && n_vec * lanes < 2L * kNumSMs * 256) lanes *= 2;
    r.lanes = lanes;
    long blocks = (n_vec + (256 / lanes) - 1) / (256 / lanes);
    if (blocks > 8L * kNumSMs) blocks = 8L * kNumSMs;
    tc::reduce_partials_kernel<<<dim3((unsigned)blocks, r.n_layers > 0 ? r.n_layers : 1), 256, 0, st>>>(r);
    return launch_status();
}

// Tile shape: 256 x 256 (MT = 2) cuts the L2->SM traffic per flop by a third but has a single
// accumulator buffer; it pays once d_out spans at least two 128-row sub-tiles.
template <int MT>
int launch_zta_tc_mt(const tc::zta::Maps& maps, tc::zta::Params p, int B, bool norm_mode,
                     float* gW, long ldg, float* gb, float* sq, int d_in, int d_out, void* workspace,
                     size_t workspace_bytes, const NoiseSpec* noise, bool* noise_done, cudaStream_t st,
                     bool fit_to_workspace = false, const GradGroup* grp = nullptr) {
    namespace z = tc::zta;
    constexpr int BM = z::Cfg<MT>::BM;
    const long R = p.R;
    p.tiles_m_layer = ceil_div(d_out, BM);
    p.tiles_m = p.tiles_m_layer * (grp && grp->n > 0 ? grp->n : 1);
    p.tiles_n = ceil_div(d_in, z::BN);
    const int tiles = p.tiles_m * p.tiles_n;
    int ksplit = 1;
    if (norm_mode) {
        p.n_items = B * tiles;
        if (cudaMemsetAsync(sq, 0, sizeof(float) * (size_t)B, st) != cudaSuccess) return DPCLIP_ERR_CUDA;
    } else {
        const int nkb = ceil_div(R, z::Cfg<MT>::BK);
        // One wave of equally long items: the kernel is bound by L2->SM traffic, so what matters is that
        // every SM streams the same number of row blocks.  (MT = 1 has two accumulator buffers and can
        // overlap the epilogue of one item with the next, so it takes two items per SM when they stay long.)
        const int sms = sm_budget();
        const int per_sm = (MT == 1 && tiles <= sms && nkb / ((2 * sms) / tiles) >= 16) ? 2 : 1;
        const ZtaSplit split = zta_pick_split(nkb, tiles, per_sm, sms);
        // the preferred split when the workspace holds its partial tiles, else one wave
        ksplit = split.one_wave;
        if (split.preferred != split.one_wave && !fit_to_workspace &&
            workspace_bytes >= kHeaderBytes + zta_scratch_bytes(tiles, split.preferred, BM, gb != nullptr))
            ksplit = split.preferred;
        if (fit_to_workspace) {                 // fixed-size scratch: take fewer, longer row slices
            const size_t per_item = (size_t)BM * z::BN * 4 + (gb ? (size_t)BM * 4 : 0);
            const size_t room = workspace_bytes > (size_t)kHeaderBytes ? workspace_bytes - kHeaderBytes : 0;
            const long fit = (long)(room / per_item / tiles);
            if (ksplit > fit) ksplit = (int)fit;
        }
        if (ksplit > nkb) ksplit = nkb;
        if (ksplit < 1) ksplit = 1;
        p.kb_per_split = ceil_div(nkb, ksplit);
        ksplit = ceil_div(nkb, p.kb_per_split);
        p.n_items = tiles * ksplit;
        if (grp && grp->n > 0 && ksplit == 1) return 1;        // a group's outputs go through the partial tiles
        if (ksplit > 1) {
            const size_t part_bytes = (size_t)p.n_items * BM * z::BN * 4;
            const size_t bias_bytes = gb ? (size_t)p.n_items * BM * 4 : 0;
            if (workspace_bytes < kHeaderBytes + part_bytes + bias_bytes) return DPCLIP_ERR_WORKSPACE;
            p.part = reinterpret_cast<float*>(static_cast<char*>(workspace) + kHeaderBytes);
            p.bias_part = gb ? p.part + part_bytes / 4 : nullptr;
        } else if (gb && cudaMemsetAsync(gb, 0, sizeof(float) * (size_t)d_out, st) != cudaSuccess) {
            return DPCLIP_ERR_CUDA;         // single item per tile: direct stores, bias by red.add
        }
    }
    if (!enable_smem(tc::zta_tc_kernel<MT>, z::SMEM_BYTES)) return DPCLIP_ERR_CUDA;
    const int grid = p.n_items < sm_budget() ? p.n_items : sm_budget();
    tc::zta_tc_kernel<MT><<<grid, z::THREADS, z::SMEM_BYTES, st>>>(maps, p);
    int rc = launch_status();
    if (rc || norm_mode || ksplit == 1) return rc;

    return launch_reduce_partials(p, tiles, ksplit, BM, z::BN, d_in, d_out, gW, ldg, gb, noise, noise_done, st, grp);
}

// Clipped sums on CTA pairs (zta_pair_kernel): 512 x 256 tiles, the (tile, stage) units of all layers of the
// launch cut into equal runs, one per pair.  A layer qualifies when the padding of d_out to 512-row pair tiles
// costs at most a tenth more than its padding to 256-row tiles.
constexpr int kNumPairs = kNumSMs / 2;
inline bool pair_tile_ok(int d_out) {
    if (path_switch(SW_NO_PAIR) || d_out <= 256) return false;
    const double pad_pair = (double)ceil_div(d_out, 512) * 512, pad_single = (double)ceil_div(d_out, 256) * 256;
    return pad_pair <= 1.1 * pad_single;
}
inline int pair_tiles(int d_in, int d_out) { return ceil_div(d_out, tc::ztp::BM) * ceil_div(d_in, tc::ztp::BN); }
inline size_t pair_segment_bytes(bool bias) {
    return tc::ztp::SEG_ELEMS * 4 + (bias ? (size_t)tc::ztp::BM * 4 : 0);
}
// scratch for a launch over `tiles` pair tiles with every pair busy: one segment per tile position of every
// super-layer (at most tiles + 15 positions when narrow layers leave a super-layer part empty) and one per pair
inline size_t pair_scratch_bytes(int tiles) { return (size_t)(tiles + 16 + kNumPairs) * pair_segment_bytes(true); }
inline long gcd_l(long a, long b) { while (b) { const long t = a % b; a = b; b = t; } return a; }

struct StreamLayer {
    const void* A; long lda; const void* Z; long ldz; int d_in, d_out;
    float* gW; long ldg; float* gb; unsigned long long sid_w, sid_b;
    const float* clip;             // this layer's factors [B], or NULL
};

// Returns DPCLIP_OK, a negative status, or 1 when the workspace cannot hold even one segment per tile (the
// caller then takes another path).
int launch_zta_stream(const StreamLayer* ls, int n, int B, int T, const NoiseSpec* noise,
                      bool* noise_done, void* workspace, size_t workspace_bytes, cudaStream_t st) {
    namespace zp = tc::ztp;
    if (n < 1 || n > zp::MAX_LAYERS) return 1;
    const long R = (long)B * T;
    tc::zta::Maps maps;
    zp::Params p;
    memset(&p, 0, sizeof(p));
    p.R = (int)R; p.T = T; p.S = (int)ceil_div(R, (long)zp::BK); p.n_layers = n;
    p.status = static_cast<int*>(workspace);
    bool fuse_noise = noise && noise->scale > 0.f;
    int G = 0;
    for (int l = 0; l < n; ++l) {
        const StreamLayer& y = ls[l];
        if (!make_map_bf16(&maps.a[l], y.A, R, y.d_in, y.lda, 64, zp::BK) ||
            !make_map_bf16(&maps.z[l], y.Z, R, y.d_out, y.ldz, 64, zp::BK))
            return DPCLIP_ERR_CUDA;
        zp::Layer& q = p.layer[l];
        q.d_in = y.d_in; q.d_out = y.d_out;
        q.tiles_n = ceil_div(y.d_in, zp::BN);
        q.tile_base = G; q.tiles = pair_tiles(y.d_in, y.d_out);
        G += q.tiles;
        q.do_bias = y.gb ? 1 : 0;
        q.clip = y.clip;
        q.gW = y.gW; q.gb = y.gb; q.ldg = y.ldg;
        q.vec_ok = aligned_to(y.gW, 16) && y.ldg % 4 == 0;
        q.sw0 = (uint32_t)y.sid_w; q.sw1 = (uint32_t)(y.sid_w >> 32);
        q.sb0 = (uint32_t)y.sid_b; q.sb1 = (uint32_t)(y.sid_b >> 32);
        if (y.gb) p.any_bias = 1;
        // the noise of element j is indexed by its position in the dense tensor, one Philox block per float4
        if (y.ldg != y.d_in || y.d_in % 4 != 0) fuse_noise = false;
    }
    p.G = G;
    if (G > zp::MAX_TILES) return 1;
    // Gang width: the widest W <= 16 for which every layer either splits into whole super-layers (tiles % W == 0)
    // or is narrower than W (narrow layers are packed side by side), and whose gangs and super-layers leave at
    // most a tenth of the pairs idle; else W = 1 (tile-major, no sharing of rows between tiles).
    int W = 1, n_super = G;
    for (int w = 16; w >= 2; --w) {
        bool ok = true;
        int supers = 0, open_fill = 0;              // narrow layers: first fit into the open super-layer
        for (int l = 0; l < n && ok; ++l) {
            const int t = p.layer[l].tiles;
            if (t >= w) { ok = t % w == 0; supers += t / w; }
            else if (open_fill > 0 && open_fill + t <= w) open_fill += t;
            else { ++supers; open_fill = t; }
        }
        if (!ok || (long)supers * w > zp::MAX_TILES) continue;
        const double use = (double)(kNumPairs / w) * w / kNumPairs * ((double)G / ((double)supers * w));
        if (use >= 0.9) { W = w; n_super = supers; break; }
    }
    p.W = W; p.n_super = n_super;
    for (int i = 0; i < zp::MAX_TILES; ++i) { p.super_tile[i] = -1; p.tile_slot[i] = 0; }
    {
        int next_super = 0, open_super = -1, open_fill = 0;
        for (int l = 0; l < n; ++l) {
            const zp::Layer& q = p.layer[l];
            if (q.tiles >= W) {
                for (int t = 0; t < q.tiles; ++t) {
                    const int sl = next_super + t / W, j = t % W;
                    p.super_tile[sl * W + j] = (short)(q.tile_base + t);
                    p.tile_slot[q.tile_base + t] = (short)(sl * W + j);
                }
                next_super += q.tiles / W;
            } else {
                if (open_super < 0 || open_fill + q.tiles > W) { open_super = next_super++; open_fill = 0; }
                for (int t = 0; t < q.tiles; ++t) {
                    p.super_tile[open_super * W + open_fill + t] = (short)(q.tile_base + t);
                    p.tile_slot[q.tile_base + t] = (short)(open_super * W + open_fill + t);
                }
                open_fill += q.tiles;
            }
        }
        if (next_super != n_super || (long)n_super * W > zp::MAX_TILES) return 1;
    }
    p.total = (long)n_super * p.S;
    // equal runs over all gangs; runs shorter than eight stages would be mostly set-up and drain
    const size_t seg_bytes = pair_segment_bytes(p.any_bias != 0);
    const size_t room = workspace && workspace_bytes > (size_t)kHeaderBytes ? workspace_bytes - kHeaderBytes : 0;
    const long max_segments = (long)(room / seg_bytes) / W;          // per gang position
    if (max_segments < n_super) return 1;
    long U = ceil_div(p.total, (long)(kNumPairs / W));
    if (U < 8) U = p.total < 8 ? p.total : 8;
    // a small workspace (the fixed array of the entry point without one) limits the number of runs
    while (zp::segment_of(p.total - 1, p.S, (int)U, (long)p.S / gcd_l(p.S, U) * U) + 1 > max_segments) {
        const long runs = ceil_div(p.total, U);
        if (runs <= 1) return 1;
        U = ceil_div(p.total, runs - 1);
    }
    p.U = (int)U;
    p.lcm = (long)p.S / gcd_l(p.S, U) * U;
    const long n_segments = (zp::segment_of(p.total - 1, p.S, p.U, p.lcm) + 1) * W;
    p.n_segments = n_segments;
    for (int t = 0; t < G; ++t) {                                   // the reduce kernel's view of the same cut
        const long sl = p.tile_slot[t] / W, j = p.tile_slot[t] % W;
        const long s0 = zp::segment_of(sl * p.S, p.S, p.U, p.lcm), s1 = zp::segment_of((sl + 1) * p.S - 1, p.S, p.U, p.lcm);
        p.seg_first[t] = (int)(s0 * W + j);
        p.seg_count[t] = (short)(s1 - s0 + 1);
    }
    for (int l = 0; l < n; ++l)
        for (int t = 0; t < p.layer[l].tiles; ++t) p.tile_layer[p.layer[l].tile_base + t] = (unsigned char)l;
    p.part = reinterpret_cast<float*>(static_cast<char*>(workspace) + kHeaderBytes);
    p.bias_part = p.any_bias ? p.part + (size_t)n_segments * zp::SEG_ELEMS : nullptr;
    if (fuse_noise) {
        p.noise_scale = noise->scale;
        p.k0 = (uint32_t)noise->seed; p.k1 = (uint32_t)(noise->seed >> 32);
        if (noise_done) *noise_done = true;
    }
    if (!enable_smem(tc::zta_pair_kernel, zp::SMEM_BYTES)) return DPCLIP_ERR_CUDA;
    const int pairs = (int)ceil_div(p.total, U) * W;
    DPCLIP_LOGF("clipped sum, CTA pairs: %d layer(s), B*T=%ld, %d tiles of 512x256 in %d super-layer(s) of %d, %d stages per tile, "
                "%d pairs in gangs of %d, runs of %ld stages, %ld segments, noise %s", n, R, G, n_super, W, p.S, pairs, W, U,
                n_segments, fuse_noise ? "in the reduce" : "separate");
    if (t_overlap_prev && !path_switch(SW_NO_OVERLAP)) {
        t_overlap_prev = false;                    // only the launch that directly follows
        cudaLaunchConfig_t cfg;
        memset(&cfg, 0, sizeof(cfg));
        cfg.gridDim = dim3(2 * pairs); cfg.blockDim = dim3(zp::THREADS);
        cfg.dynamicSmemBytes = zp::SMEM_BYTES; cfg.stream = st;
        cudaLaunchAttribute attr[1];
        attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
        attr[0].val.programmaticStreamSerializationAllowed = 1;
        cfg.attrs = attr; cfg.numAttrs = 1;
        if (cudaLaunchKernelEx(&cfg, tc::zta_pair_kernel, maps, p) != cudaSuccess) { cudaGetLastError(); return DPCLIP_ERR_CUDA; }
    } else {
        tc::zta_pair_kernel<<<2 * pairs, zp::THREADS, zp::SMEM_BYTES, st>>>(maps, p);
    }
    int rc = launch_status();
    if (rc) return rc;
    // one wave of CTAs (six of 256 threads and 40 registers per SM) over the 4-row blocks of all tiles
    long blocks = (long)G * (zp::BM / 4);
    if (blocks > 6L * kNumSMs) blocks = 6L * kNumSMs;
    tc::reduce_segments_kernel<<<(unsigned)blocks, 256, 0, st>>>(p);
    return launch_status();
}

int launch_zta_tc(const void* A, long lda, const void* Z, long ldz, int B, int T, int d_in, int d_out,
                  bool norm_mode, int has_bias, const float* clip, float* gW, long ldg, float* gb, float* sq,
                  void* workspace, size_t workspace_bytes, const NoiseSpec* noise, bool* noise_done,
                  cudaStream_t st, bool fit_to_workspace = false) {
    namespace z = tc::zta;
    const long R = (long)B * T;
    int mt = d_out > 128 ? 2 : 1;
    if (path_switch(SW_TILE_M1)) mt = 1;
    if (path_switch(SW_TILE_M2)) mt = 2;
    const bool pair = !norm_mode && mt == 2 && pair_tile_ok(d_out);
    const int bk = mt == 2 ? z::Cfg<2>::BK : z::Cfg<1>::BK;           // rows of a TMA box = rows of a stage
    z::Maps maps;
    if (!make_map_bf16(&maps.a[0], A, R, d_in, lda, 64, bk) || !make_map_bf16(&maps.z[0], Z, R, d_out, ldz, 64, bk))
        return DPCLIP_ERR_CUDA;
    z::Params p;
    memset(&p, 0, sizeof(p));
    p.R = (int)R; p.T = T; p.d_in = d_in; p.d_out = d_out;
    p.norm_mode = norm_mode ? 1 : 0;
    p.status = static_cast<int*>(workspace);
    if (norm_mode) {
        p.do_bias = has_bias ? 1 : 0;
        p.sq = sq;
    } else {
        p.clip = clip; p.gW = gW; p.ldg = ldg; p.gb = gb;
        p.do_bias = gb ? 1 : 0;
        p.vec_ok = aligned_to(gW, 16) && ldg % 4 == 0;
    }
    if (pair) {
        const StreamLayer one = {A, lda, Z, ldz, d_in, d_out, gW, ldg, gb, noise ? noise->sid_w : 0ull, noise ? noise->sid_b : 0ull, clip};
        const int rc = launch_zta_stream(&one, 1, B, T, noise, noise_done, workspace, workspace_bytes, st);
        if (rc <= 0) return rc;                 // 1: not even one segment per tile fits -> the single-CTA kernel below
    }
    if (mt == 2)
        return launch_zta_tc_mt<2>(maps, p, B, norm_mode, gW, ldg, gb, sq, d_in, d_out, workspace, workspace_bytes,
                                   noise, noise_done, st, fit_to_workspace);
    return launch_zta_tc_mt<1>(maps, p, B, norm_mode, gW, ldg, gb, sq, d_in, d_out, workspace, workspace_bytes,
                               noise, noise_done, st, fit_to_workspace);
}

// Clipped sums (+ noise) of n layers of ONE shape in one tensor-core launch and one reduce launch.
// Returns 1 when the group does not qualify (the caller then goes layer by layer).
int launch_zta_tc_group(const dpclip_layer* const* ls, const int* index, int n, int B, const float* clip,
                        float noise_scale, unsigned long long seed, unsigned long long stream_id0,
                        void* workspace, size_t workspace_bytes, cudaStream_t st) {
    namespace z = tc::zta;
    if (n < 2 || n > z::MAX_LAYERS) return 1;
    const dpclip_layer& y0 = *ls[0];
    const long R = (long)B * y0.T;
    const int bk = y0.d_out > 128 ? z::Cfg<2>::BK : z::Cfg<1>::BK;
    z::Maps maps;
    GradGroup grp;
    memset(&grp, 0, sizeof(grp));
    grp.n = n;
    float* any_gb = nullptr;
    bool vec_ok = true;
    for (int l = 0; l < n; ++l) {
        const dpclip_layer& y = *ls[l];
        if (!make_map_bf16(&maps.a[l], y.A, R, y.d_in, y.lda, 64, bk) ||
            !make_map_bf16(&maps.z[l], y.Zbar, R, y.d_out, y.ldz, 64, bk))
            return DPCLIP_ERR_CUDA;
        grp.gW[l] = y.gW; grp.gb[l] = y.has_bias ? y.gb : nullptr;
        grp.sid_w[l] = stream_id0 + 2ull * index[l]; grp.sid_b[l] = grp.sid_w[l] + 1;
        if (grp.gb[l]) any_gb = grp.gb[l];
        vec_ok = vec_ok && aligned_to(y.gW, 16);
    }
    z::Params p;
    memset(&p, 0, sizeof(p));
    p.R = (int)R; p.T = y0.T; p.d_in = y0.d_in; p.d_out = y0.d_out;
    p.status = static_cast<int*>(workspace);
    p.clip = clip; p.gW = y0.gW; p.ldg = y0.d_in; p.gb = any_gb;
    p.do_bias = any_gb ? 1 : 0;
    p.vec_ok = vec_ok && y0.d_in % 4 == 0;
    const NoiseSpec ns = {noise_scale, seed, 0, 0};             // the streams come from the group
    bool noise_done = false;
    int rc;
    if (y0.d_out > 128)
        rc = launch_zta_tc_mt<2>(maps, p, B, false, y0.gW, y0.d_in, any_gb, nullptr, y0.d_in, y0.d_out, workspace,
                                 workspace_bytes, &ns, &noise_done, st, false, &grp);
    else
        rc = launch_zta_tc_mt<1>(maps, p, B, false, y0.gW, y0.d_in, any_gb, nullptr, y0.d_in, y0.d_out, workspace,
                                 workspace_bytes, &ns, &noise_done, st, false, &grp);
    if (rc) return rc;
    if (noise_scale > 0.f && !noise_done) return DPCLIP_ERR_UNSUPPORTED;     // the caller checked d_in % 4
    return DPCLIP_OK;
}

// fp32 layers on the tensor cores (error-compensated tf32): TMA needs 16-byte aligned bases and rows
inline bool tf32_eligible(const void* A, long lda, const void* Z, long ldz, int B, int T, int d_in, int d_out,
                          dpclip_dtype dtype) {
    if (dtype != DPCLIP_F32) return false;
    if (path_switch(SW_FORCE_SIMT)) return false;
    if (!(aligned_to(A, 16) && aligned_to(Z, 16) && lda % 4 == 0 && ldz % 4 == 0)) return false;
    // worth it once there is real contraction work; tiny layers stay on the fp32-ALU kernels
    return (double)B * T * d_in * d_out >= 32.0 * 1024 * 1024;
}

bool make_map_f32(CUtensorMap* map, const void* base, long rows, long cols, long ld, int box_cols, int box_rows) {
    EncodeTiledFn fn = encode_tiled_fn();
    if (!fn) return false;
    cuuint64_t dims[2] = {(cuuint64_t)cols, (cuuint64_t)rows};
    cuuint64_t strides[1] = {(cuuint64_t)ld * 4};
    cuuint32_t box[2] = {(cuuint32_t)box_cols, (cuuint32_t)box_rows};
    cuuint32_t estr[2] = {1, 1};
    return fn(map, CU_TENSOR_MAP_DATA_TYPE_FLOAT32, 2, const_cast<void*>(base), dims, strides, box, estr,
              CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B_ATOM_32B,
              CU_TENSOR_MAP_L2_PROMOTION_L2_256B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

int launch_zta_tf32(const void* A, long lda, const void* Z, long ldz, int B, int T, int d_in, int d_out,
                    bool norm_mode, int has_bias, const float* clip, float* gW, long ldg, float* gb, float* sq,
                    void* workspace, size_t workspace_bytes, const NoiseSpec* noise, bool* noise_done,
                    cudaStream_t st, const tc::ConvGather* conv = nullptr) {
    namespace t = tc::t32;
    const long R = (long)B * T;
    CUtensorMap ma, mz;
    if (!make_map_f32(&mz, Z, R, d_out, ldz, 32, t::BK)) return DPCLIP_ERR_CUDA;
    if (conv) ma = mz;                                       // A is gathered from the feature map: no tensor map for it
    else if (!make_map_f32(&ma, A, R, d_in, lda, 32, t::BK)) return DPCLIP_ERR_CUDA;
    tc::zta::Params p;
    memset(&p, 0, sizeof(p));
    p.R = (int)R; p.T = T; p.d_in = d_in; p.d_out = d_out;
    p.norm_mode = norm_mode ? 1 : 0;
    p.status = static_cast<int*>(workspace);
    p.tiles_m = ceil_div(d_out, t::BM); p.tiles_n = ceil_div(d_in, t::BN);
    const int tiles = p.tiles_m * p.tiles_n;
    int ksplit = 1;
    if (norm_mode) {
        p.do_bias = has_bias ? 1 : 0;
        p.sq = sq;
        p.n_items = B * tiles;
        if (cudaMemsetAsync(sq, 0, sizeof(float) * (size_t)B, st) != cudaSuccess) return DPCLIP_ERR_CUDA;
    } else {
        p.clip = clip; p.gW = gW; p.ldg = ldg; p.gb = gb;
        p.do_bias = gb ? 1 : 0;
        p.vec_ok = aligned_to(gW, 16) && ldg % 4 == 0;
        const int nkb = ceil_div(R, t::BK);
        // two accumulator buffers: two items per SM when they stay long enough, else one wave
        const int sms = sm_budget();
        const int per_sm = (tiles <= sms && nkb / ((2 * sms) / tiles) >= 16) ? 2 : 1;
        ksplit = (per_sm * sms) / tiles;
        if (ksplit > nkb) ksplit = nkb;
        if (ksplit < 1) ksplit = 1;
        p.kb_per_split = ceil_div(nkb, ksplit);
        ksplit = ceil_div(nkb, p.kb_per_split);
        p.n_items = tiles * ksplit;
        if (ksplit > 1) {
            const size_t part_bytes = (size_t)p.n_items * t::BM * t::BN * 4;
            const size_t bias_bytes = gb ? (size_t)p.n_items * t::BM * 4 : 0;
            if (workspace_bytes < kHeaderBytes + part_bytes + bias_bytes) return DPCLIP_ERR_WORKSPACE;
            p.part = reinterpret_cast<float*>(static_cast<char*>(workspace) + kHeaderBytes);
            p.bias_part = gb ? p.part + part_bytes / 4 : nullptr;
        } else if (gb && cudaMemsetAsync(gb, 0, sizeof(float) * (size_t)d_out, st) != cudaSuccess) {
            return DPCLIP_ERR_CUDA;
        }
    }
    const int grid = p.n_items < sm_budget() ? p.n_items : sm_budget();
    if (conv) {
        if (!enable_smem(tc::zta_tf32_kernel<true>, t::SMEM_BYTES)) return DPCLIP_ERR_CUDA;
        tc::zta_tf32_kernel<true><<<grid, t::THREADS, t::SMEM_BYTES, st>>>(ma, mz, p, *conv);
    } else {
        tc::ConvGather none;
        memset(&none, 0, sizeof(none));
        if (!enable_smem(tc::zta_tf32_kernel<false>, t::SMEM_BYTES)) return DPCLIP_ERR_CUDA;
        tc::zta_tf32_kernel<false><<<grid, t::THREADS, t::SMEM_BYTES, st>>>(ma, mz, p, none);
    }
    int rc = launch_status();
    if (rc || norm_mode || ksplit == 1) return rc;
    return launch_reduce_partials(p, tiles, ksplit, t::BM, t::BN, d_in, d_out, gW, ldg, gb, noise, noise_done, st);
}

// clipped sum of one layer, optionally with the noise folded into the last pass over the output
int clipped_grad_impl(const void* A, long lda, const void* Zbar, long ldz, int B, int T, int d_in, int d_out,
                      dpclip_dtype dtype, const float* clip, float* gW, long ldg, float* gb, void* workspace,
                      size_t workspace_bytes, const NoiseSpec* noise, bool* noise_done, cudaStream_t st) {
    DPCLIP_LOGF("clipped_grad B=%d T=%d %d->%d %s: %s", B, T, d_in, d_out, dtype == DPCLIP_F32 ? "f32" : "bf16",
                tc_eligible(A, lda, Zbar, ldz, dtype) ? "tcgen05 bf16"
                : (tf32_eligible(A, lda, Zbar, ldz, B, T, d_in, d_out, dtype) && !narrow_layer(T, d_in, d_out, gb != nullptr, lda, ldz))
                      ? "tcgen05 3xtf32" : "fp32-ALU / narrow kernels");
    if (tc_eligible(A, lda, Zbar, ldz, dtype))
        return launch_zta_tc(A, lda, Zbar, ldz, B, T, d_in, d_out, false, 0, clip, gW, ldg, gb, nullptr, workspace,
                             workspace_bytes, noise, noise_done, st);
    if (tf32_eligible(A, lda, Zbar, ldz, B, T, d_in, d_out, dtype) && !narrow_layer(T, d_in, d_out, gb != nullptr, lda, ldz))
        return launch_zta_tf32(A, lda, Zbar, ldz, B, T, d_in, d_out, false, 0, clip, gW, ldg, gb, nullptr, workspace,
                               workspace_bytes, noise, noise_done, st);
    return launch_simt_grad(A, lda, Zbar, ldz, B, T, d_in, d_out, dtype, clip, gW, ldg, gb, st, workspace,
                            workspace_bytes, noise, noise_done);
}


// Whole step in two launches for models made of T = 1 layers only (see kernels_fused_t1.cuh).
// Returns 1 when the fused path does not apply (the caller then takes the per-layer path).
// Second launch of the fused step on the tensor cores (fp32 models).  Every layer must either be addressable
// by TMA (16-byte aligned base and row stride); the zb of a thin layer (at most 16 outputs) need not be.  Returns 1 when the model
// does not qualify, so that the caller falls back to the fp32-ALU kernel.
// Alignment that TMA asks of one operand of the fused tensor-core kernels (16-byte base and row stride).
inline bool t1_tma_ok(const void* ptr, long ld, dpclip_dtype dtype) {
    return aligned_to(ptr, 16) && ld % (dtype == DPCLIP_BF16 ? 8 : 4) == 0;
}

template <typename T>
int launch_fused_t1_tc(tc::f1::Params& q, bool one_launch, int grid, void* workspace, cudaStream_t st) {
    namespace f = tc::f1;
    if (one_launch) {
        // the whole step as one cooperative launch (its CTAs meet at a grid-wide barrier)
        q.grid_counter = reinterpret_cast<unsigned int*>(static_cast<char*>(workspace) + kGridCounterOffset);
        if (!enable_smem(tc::t1_all_grads_tf32_kernel<true, T>, f::SMEM_BYTES)) return DPCLIP_ERR_CUDA;
        cudaLaunchConfig_t cfg;
        memset(&cfg, 0, sizeof(cfg));
        cfg.gridDim = dim3(grid); cfg.blockDim = dim3(f::THREADS); cfg.dynamicSmemBytes = f::SMEM_BYTES; cfg.stream = st;
        cudaLaunchAttribute attr;
        attr.id = cudaLaunchAttributeCooperative; attr.val.cooperative = 1;
        cfg.attrs = &attr; cfg.numAttrs = 1;
        if (cudaLaunchKernelEx(&cfg, tc::t1_all_grads_tf32_kernel<true, T>, q) != cudaSuccess) {
            cudaGetLastError();
            return 1;                       // cannot be made resident at once: take the two-launch form
        }
        return launch_status();
    }
    if (!enable_smem(tc::t1_all_grads_tf32_kernel<false, T>, f::SMEM_BYTES)) return DPCLIP_ERR_CUDA;
    tc::t1_all_grads_tf32_kernel<false, T><<<grid, f::THREADS, f::SMEM_BYTES, st>>>(q);
    return launch_status();
}

int launch_fused_t1_tf32(const FusedT1Params& base, bool one_launch, dpclip_dtype dtype, void* workspace,
                         size_t workspace_bytes, cudaStream_t st) {
    namespace f = tc::f1;
    if (path_switch(SW_NO_T1_TF32)) return 1;
    if (!workspace || workspace_bytes < kHeaderBytes) return 1;
    static_assert(sizeof(f::Params) <= 4096, "kernel parameter space");
    f::Params q;
    memset(&q, 0, sizeof(q));
    q.base = base;
    q.status = static_cast<int*>(workspace);
    const bool bf16 = dtype == DPCLIP_BF16;
    int items = 0, tc_layers = 0;
    for (int l = 0; l < base.L; ++l) {
        const FusedT1Layer& y = base.layer[l];
        const bool thin = y.d_out <= f::THIN_MAX_OUT;
        if (!t1_tma_ok(y.A, y.lda, dtype) || !(t1_tma_ok(y.Z, y.ldz, dtype) || thin)) return 1;
        q.item_begin[l] = items;
        q.thin[l] = thin ? 1 : 0;
        if (bf16) {
            if (!make_map_bf16(&q.map_a[l], y.A, base.B, y.d_in, y.lda, 64, f::BK)) return DPCLIP_ERR_CUDA;
            if (!thin && !make_map_bf16(&q.map_z[l], y.Z, base.B, y.d_out, y.ldz, 64, f::BK)) return DPCLIP_ERR_CUDA;
        } else {
            if (!make_map_f32(&q.map_a[l], y.A, base.B, y.d_in, y.lda, 32, f::BK)) return DPCLIP_ERR_CUDA;
            if (!thin && !make_map_f32(&q.map_z[l], y.Z, base.B, y.d_out, y.ldz, 32, f::BK)) return DPCLIP_ERR_CUDA;
        }
        q.tiles_n[l] = ceil_div(y.d_in, f::BN);
        items += ceil_div(y.d_out, f::BM) * q.tiles_n[l];
        if (!thin) ++tc_layers;
    }
    if (!tc_layers) return 1;
    q.total_items = items;
    const int grid = items < kNumSMs ? items : kNumSMs;
    return bf16 ? launch_fused_t1_tc<__nv_bfloat16>(q, one_launch, grid, workspace, st)
                : launch_fused_t1_tc<float>(q, one_launch, grid, workspace, st);
}

// One T = 1 layer of the caller's model as the fused kernels see it.  Returns 0, 1 (the layer does not
// qualify for the fused kernels) or a negative argument error.
int fill_fused_t1_layer(FusedT1Layer& f, const dpclip_layer& y, int index, int B, dpclip_dtype dtype, int tile,
                        int& tiles) {
    if (y.T != 1 || y.ldg != y.d_in) return 1;
    if (y.method != DPCLIP_AUTO && y.method != DPCLIP_T1) return 1;
    int rc = check_layer_args(y.A, y.lda, y.Zbar, y.ldz, B, 1, y.d_in, y.d_out, dtype);
    if (rc) return rc;
    if (!y.gW || (y.has_bias && !y.gb)) return DPCLIP_ERR_INVALID_ARG;
    if (!aligned_to(y.gW, 16) || (y.gb && !aligned_to(y.gb, 4))) return 1;
    f.A = y.A; f.lda = y.lda; f.Z = y.Zbar; f.ldz = y.ldz;
    f.d_in = y.d_in; f.d_out = y.d_out; f.has_bias = y.has_bias ? 1 : 0;
    f.vec_a = vec4_ok(y.A, y.lda, dtype); f.vec_z = vec4_ok(y.Zbar, y.ldz, dtype);
    f.gW = y.gW; f.gb = y.has_bias ? y.gb : nullptr;
    f.tiles_m = ceil_div(y.d_out, tile); f.tiles_n = ceil_div(y.d_in + f.has_bias, tile);
    f.tile_begin = tiles;
    f.index = index;
    tiles += f.tiles_m * f.tiles_n;
    return 0;
}

// The T = 1 layers of a model that also has T > 1 layers (fp32): their norms in one launch (into their rows
// of sq), and, once the factors of the whole model exist, their clipped sums with noise in one tensor-core
// launch.  `group` lists the layers' positions in the model.  prepare returns 0 when the group qualifies.
struct T1Group {
    FusedT1Params p;
    bool active = false;
};

int prepare_t1_group(T1Group& g, const dpclip_layer* layers, int L, int B, dpclip_dtype dtype, float C, float sigma,
                     unsigned long long seed, unsigned long long stream_id0, float* sq, const float* clip,
                     bool mixed_only = true) {
    g.active = false;
    if (B > FUSED_MAX_B) return 0;
    if (path_switch(SW_NO_FUSED_T1)) return 0;
    if (path_switch(SW_NO_T1_TF32)) return 0;
    memset(&g.p, 0, sizeof(g.p));
    int n = 0, tiles = 0, wide = 0;
    for (int l = 0; l < L; ++l) {
        if (layers[l].T != 1) continue;
        if (n == FUSED_MAX_LAYERS) return 0;
        const int rc = fill_fused_t1_layer(g.p.layer[n], layers[l], l, B, dtype, 64, tiles);
        if (rc < 0) return rc;
        if (rc) return 0;
        const FusedT1Layer& y = g.p.layer[n];
        if (!t1_tma_ok(y.A, y.lda, dtype) || !(t1_tma_ok(y.Z, y.ldz, dtype) || y.d_out <= tc::f1::THIN_MAX_OUT))
            return 0;
        if (y.d_out > tc::f1::THIN_MAX_OUT) ++wide;
        ++n;
    }
    if (n == 0 || wide == 0 || (mixed_only && n == L)) return 0;    // the kernel wants one tensor-core layer
    g.p.L = n; g.p.B = B; g.p.total_tiles = tiles;
    g.p.C = C; g.p.noise_scale = sigma * C;
    g.p.k0 = (uint32_t)seed; g.p.k1 = (uint32_t)(seed >> 32); g.p.stream_id0 = stream_id0;
    g.p.sq = sq; g.p.clip = nullptr; g.p.norms = nullptr; g.p.clip_in = clip;
    g.active = true;
    return 0;
}

int try_fused_t1_step(const dpclip_layer* layers, int L, int B, dpclip_dtype dtype, float C, float sigma,
                      unsigned long long seed, unsigned long long stream_id0, float* sq, float* clip,
                      float* norms, void* workspace, size_t workspace_bytes, cudaStream_t st) {
    if (L > FUSED_MAX_LAYERS || B > FUSED_MAX_B) return 1;
    if (path_switch(SW_NO_FUSED_T1)) return 1;
    FusedT1Params p;
    memset(&p, 0, sizeof(p));
    // fp32-ALU form: 64 x 64 tiles, several CTAs per SM hide the global-load latency of these short (K = B)
    // products (128 x 128 register tiles, one CTA per SM, measured slower: 61 vs 39 us per step on the
    // 784-1000-1000-10, B = 128 model).
    const int tile = 64;
    int tiles = 0;
    for (int l = 0; l < L; ++l) {
        const int rc = fill_fused_t1_layer(p.layer[l], layers[l], l, B, dtype, tile, tiles);
        if (rc) return rc;
    }
    p.L = L; p.B = B; p.total_tiles = tiles;
    p.C = C; p.noise_scale = sigma * C;
    p.k0 = (uint32_t)seed; p.k1 = (uint32_t)(seed >> 32); p.stream_id0 = stream_id0;
    p.sq = sq; p.clip = clip; p.norms = norms;
    const int rows = L * B;
    const int grid_n = rows;
    const int grid_g = tiles < 4 * kNumSMs ? tiles : 4 * kNumSMs;
    const int smem64 = FusedT1Cfg<64>::SMEM_BYTES;
    bool one = true;
    if (path_switch(SW_T1_TWO_LAUNCHES)) one = false;
    if (one) {
        const int rc = launch_fused_t1_tf32(p, true, dtype, workspace, workspace_bytes, st);
        if (rc <= 0) return rc;
    }
    if (dtype == DPCLIP_F32) t1_all_norms_kernel<float><<<grid_n, 128, 0, st>>>(p);
    else t1_all_norms_kernel<__nv_bfloat16><<<grid_n, 128, 0, st>>>(p);
    if (launch_status()) return DPCLIP_ERR_CUDA;
    const int rc = launch_fused_t1_tf32(p, false, dtype, workspace, workspace_bytes, st);
    if (rc <= 0) return rc;
    if (dtype == DPCLIP_F32) t1_all_grads_kernel<float, 64><<<grid_g, SIMT_THREADS, smem64, st>>>(p);
    else t1_all_grads_kernel<__nv_bfloat16, 64><<<grid_g, SIMT_THREADS, smem64, st>>>(p);
    return launch_status();
}

}  // namespace

extern "C" {

int dpclip_version(void) { return 100; }
int dpclip_debug_build(void) {
#ifdef DPCLIP_DEBUG
    return 1;
#else
    return 0;
#endif
}

// An empty kernel with the launch shape of the one-launch T = 1 step: what a launch costs before it computes.
__global__ void null_launch_kernel(int* sink) { if (sink && threadIdx.x == 0xFFFFFF) *sink = 0; }

int dpclip_null_launch(int cooperative, int grid, void* stream) {
    namespace f = tc::f1;
    if (grid < 1 || grid > kNumSMs) return DPCLIP_ERR_INVALID_ARG;
    if (!enable_smem(null_launch_kernel, f::SMEM_BYTES)) return DPCLIP_ERR_CUDA;
    cudaLaunchConfig_t cfg;
    memset(&cfg, 0, sizeof(cfg));
    cfg.gridDim = dim3(grid); cfg.blockDim = dim3(f::THREADS); cfg.dynamicSmemBytes = f::SMEM_BYTES;
    cfg.stream = (cudaStream_t)stream;
    cudaLaunchAttribute attr;
    attr.id = cudaLaunchAttributeCooperative; attr.val.cooperative = cooperative ? 1 : 0;
    cfg.attrs = &attr; cfg.numAttrs = 1;
    int* none = nullptr;
    if (cudaLaunchKernelEx(&cfg, null_launch_kernel, none) != cudaSuccess) { cudaGetLastError(); return DPCLIP_ERR_CUDA; }
    return launch_status();
}

unsigned long long dpclip_launch_count(void) { return g_launches.load(std::memory_order_relaxed); }
void dpclip_reload_path_switches(void) { read_path_switches(); }

#ifdef DPCLIP_TRACE
int dpclip_trace_copy(unsigned long long* host) {
    return cudaMemcpyFromSymbol(host, tc::g_trace, sizeof(unsigned long long) * 148 * 4 * 256) == cudaSuccess ? 0 : -5;
}
#endif

const char* dpclip_status_string(int status) {
    switch (status) {
        case DPCLIP_OK: return "ok";
        case DPCLIP_ERR_INVALID_ARG: return "invalid argument";
        case DPCLIP_ERR_UNSUPPORTED: return "method not supported for this dtype/shape/alignment";
        case DPCLIP_ERR_MISALIGNED: return "pointer not aligned to its element size";
        case DPCLIP_ERR_WORKSPACE: return "workspace missing or too small";
        case DPCLIP_ERR_CUDA: return "CUDA call or kernel launch failed";
        case DPCLIP_ERR_TIMEOUT: return "a bounded device-side wait ran out";
        case DPCLIP_ERR_RANGE: return "range-checked build: an index left its buffer (access skipped)";
        default: return "unknown status";
    }
}

int dpclip_pick_method(int B, int T, int d_in, int d_out, long lda, long ldz, dpclip_dtype dtype) {
    (void)B;
    if (T == 1) return DPCLIP_T1;
    // alignment of the base pointers is not known here; rows must be 16-byte multiples for TMA
    if (dtype == DPCLIP_BF16 && lda % 8 == 0 && ldz % 8 == 0) {
        if (!path_switch(SW_FORCE_SIMT)) {
            const double gram = (double)T * (T + 1.0) * ((double)d_in + d_out);      // symmetric Gram blocks
            const double mat = 2.0 * T * (double)d_in * d_out;                       // one Zb_i^T A_i product
            return gram <= mat ? DPCLIP_GRAM : DPCLIP_MATERIALIZE;
        }
    }
    // fp32: materialised tiles on the tensor cores (error-compensated tf32) once the layer is large
    // enough and its rows are 16-byte multiples; narrow and small layers stay on the fp32 ALUs
    if (dtype == DPCLIP_F32 && lda % 4 == 0 && ldz % 4 == 0 && !narrow_layer(T, d_in, d_out, 1, lda, ldz) &&
        (double)B * T * d_in * d_out >= 32.0 * 1024 * 1024) {
        if (!path_switch(SW_FORCE_SIMT)) return DPCLIP_MATERIALIZE;
    }
    return DPCLIP_SIMT;
}

// The least workspace an entry point accepts for a layer (the public query may ask for more: see there).
static size_t workspace_floor(int B, int T, int d_in, int d_out, dpclip_dtype dtype) {
    if (dtype == DPCLIP_BF16) return kHeaderBytes + kTcScratchBytes;
    if ((double)B * T * d_in * d_out >= 32.0 * 1024 * 1024) return kHeaderBytes + kTcScratchBytes;
    return (size_t)kHeaderBytes;
}

size_t dpclip_workspace_bytes(int B, int T, int d_in, int d_out, dpclip_dtype dtype, dpclip_method method) {
    (void)method;
    // Layers that may take a tensor-core clipped sum (all bf16 layers; fp32 layers above the size where
    // the tf32 path is used) split their rows over CTAs and keep one partial tile per CTA in the
    // workspace; the bound does not depend on the layer's shape.
    if (dtype == DPCLIP_BF16) {
        // ... except for long layers whose tiles do not fill one wave of SMs: room for their preferred split
        size_t need = kTcScratchBytes;
        if (d_out > 128 && B > 0 && T > 0 && d_in > 0) {
            const int tiles = ceil_div(d_out, 256) * ceil_div(d_in, 256);
            const ZtaSplit split = zta_pick_split(ceil_div((long)B * T, 64L), tiles, 1);
            const size_t pref = zta_scratch_bytes(tiles, split.preferred, 256, true);
            if (split.preferred != split.one_wave && pref > need) need = pref;
            if (pair_tile_ok(d_out)) {                 // the CTA-pair kernel: one segment per tile and one per pair
                const size_t pneed = pair_scratch_bytes(pair_tiles(d_in, d_out));
                if (pneed > need) need = pneed;
            }
        }
        return kHeaderBytes + need;
    }
    if ((double)B * T * d_in * d_out >= 32.0 * 1024 * 1024) return kHeaderBytes + kTcScratchBytes;
    return (size_t)kHeaderBytes;
}

size_t dpclip_step_workspace_bytes(const dpclip_layer* layers, int L, int B, dpclip_dtype dtype) {
    size_t ws = kHeaderBytes;
    if (!layers || L <= 0 || B <= 0) return ws;
    for (int l = 0; l < L; ++l) {
        const dpclip_layer& y = layers[l];
        if (y.T <= 0) continue;
        const size_t w = dpclip_workspace_bytes(B, y.T, y.d_in, y.d_out, dtype, (dpclip_method)y.method);
        if (w > ws) ws = w;
    }
    if (dtype != DPCLIP_BF16 || path_switch(SW_NO_GRAD_GROUP)) return ws;
    // layers of one T that share a CTA-pair launch (up to eight): one segment per tile of all of them + one per pair
    for (int l0 = 0; l0 < L; ++l0) {
        const dpclip_layer& y0 = layers[l0];
        if (y0.T <= 1 || !pair_tile_ok(y0.d_out)) continue;
        bool first = true;
        for (int l = 0; l < l0; ++l) first = first && !(layers[l].T == y0.T && pair_tile_ok(layers[l].d_out));
        if (!first) continue;
        int n = 0, tiles = 0;
        for (int l = l0; l < L; ++l) {
            if (layers[l].T != y0.T || !pair_tile_ok(layers[l].d_out)) continue;
            tiles += pair_tiles(layers[l].d_in, layers[l].d_out);
            if (++n == tc::ztp::MAX_LAYERS) {
                if (kHeaderBytes + pair_scratch_bytes(tiles) > ws) ws = kHeaderBytes + pair_scratch_bytes(tiles);
                n = 0; tiles = 0;
            }
        }
        if (n >= 2 && kHeaderBytes + pair_scratch_bytes(tiles) > ws) ws = kHeaderBytes + pair_scratch_bytes(tiles);
    }
    return ws;
}

int dpclip_workspace_init(void* workspace, size_t workspace_bytes, void* stream) {
    if (!workspace || workspace_bytes < (size_t)kHeaderBytes) return DPCLIP_ERR_WORKSPACE;
    return cudaMemsetAsync(workspace, 0, kHeaderBytes, (cudaStream_t)stream) == cudaSuccess ? DPCLIP_OK
                                                                                             : DPCLIP_ERR_CUDA;
}

int dpclip_read_status(const void* workspace, int* host_status, void* stream) {
    if (!workspace || !host_status) return DPCLIP_ERR_INVALID_ARG;
    cudaStream_t st = (cudaStream_t)stream;
    if (cudaMemcpyAsync(host_status, workspace, sizeof(int), cudaMemcpyDeviceToHost, st) != cudaSuccess)
        return DPCLIP_ERR_CUDA;
    return cudaStreamSynchronize(st) == cudaSuccess ? DPCLIP_OK : DPCLIP_ERR_CUDA;
}

int dpclip_layer_sqnorms(const void* A, long lda, const void* Zbar, long ldz, int B, int T, int d_in,
                         int d_out, dpclip_dtype dtype, int has_bias, dpclip_method method, float* sq_layer,
                         void* workspace, size_t workspace_bytes, void* stream) {
    int rc = check_layer_args(A, lda, Zbar, ldz, B, T, d_in, d_out, dtype);
    if (rc) return rc;
    if (!sq_layer) return DPCLIP_ERR_INVALID_ARG;
    if (!aligned_to(sq_layer, 4)) return DPCLIP_ERR_MISALIGNED;
    if (method == DPCLIP_AUTO) {
        method = (dpclip_method)dpclip_pick_method(B, T, d_in, d_out, lda, ldz, dtype);
        if (dtype == DPCLIP_BF16 && (method == DPCLIP_GRAM || method == DPCLIP_MATERIALIZE) &&
            !tc_eligible(A, lda, Zbar, ldz, dtype))
            method = DPCLIP_SIMT;
        if (dtype == DPCLIP_F32 && method == DPCLIP_MATERIALIZE && !tf32_eligible(A, lda, Zbar, ldz, B, T, d_in, d_out, dtype))
            method = DPCLIP_SIMT;
    }
    if (!workspace || workspace_bytes < workspace_floor(B, T, d_in, d_out, dtype))
        return DPCLIP_ERR_WORKSPACE;
    cudaStream_t st = (cudaStream_t)stream;
    DPCLIP_LOGF("layer_sqnorms B=%d T=%d %d->%d %s bias=%d: %s", B, T, d_in, d_out, dtype == DPCLIP_F32 ? "f32" : "bf16",
                has_bias, method == DPCLIP_T1 ? "T1 closed form" : method == DPCLIP_SIMT ? "materialise, fp32-ALU / narrow kernels"
                : method == DPCLIP_GRAM ? "Gram, tcgen05" : "materialise, tcgen05");
    switch (method) {
        case DPCLIP_T1:
            if (T != 1) return DPCLIP_ERR_UNSUPPORTED;
            return launch_t1_norms(A, lda, Zbar, ldz, B, d_in, d_out, dtype, has_bias, sq_layer, st);
        case DPCLIP_SIMT:
            return launch_simt_norms(A, lda, Zbar, ldz, B, T, d_in, d_out, dtype, has_bias, sq_layer, st,
                                     static_cast<int*>(workspace));
        case DPCLIP_GRAM:
        case DPCLIP_MATERIALIZE:
            if (dtype == DPCLIP_F32) {                    // fp32: materialised tiles via error-compensated tf32
                if (method != DPCLIP_MATERIALIZE || !aligned_to(A, 16) || !aligned_to(Zbar, 16) || lda % 4 || ldz % 4)
                    return DPCLIP_ERR_UNSUPPORTED;
                return launch_zta_tf32(A, lda, Zbar, ldz, B, T, d_in, d_out, true, has_bias, nullptr, nullptr, 0,
                                       nullptr, sq_layer, workspace, workspace_bytes, nullptr, nullptr, st);
            }
            if (!aligned_to(A, 16) || !aligned_to(Zbar, 16) || lda % 8 || ldz % 8)
                return DPCLIP_ERR_UNSUPPORTED;
            if (method == DPCLIP_GRAM)
                return launch_gram_norms(A, lda, Zbar, ldz, B, T, d_in, d_out, has_bias, sq_layer,
                                         (int*)workspace, st);
            return launch_zta_tc(A, lda, Zbar, ldz, B, T, d_in, d_out, true, has_bias, nullptr, nullptr, 0,
                                 nullptr, sq_layer, workspace, workspace_bytes, nullptr, nullptr, st);
        default:
            return DPCLIP_ERR_INVALID_ARG;
    }
}

static int gram_layers_sqnorms(const dpclip_layer* layers, int L, int B, dpclip_dtype dtype, float* sq_layers,
                               int* taken, void* workspace, size_t workspace_bytes, void* stream,
                               const tc::gram::FactorsTail* tail, bool* tail_done);

int dpclip_gram_layers_sqnorms(const dpclip_layer* layers, int L, int B, dpclip_dtype dtype, float* sq_layers,
                               int* taken, void* workspace, size_t workspace_bytes, void* stream) {
    return gram_layers_sqnorms(layers, L, B, dtype, sq_layers, taken, workspace, workspace_bytes, stream, nullptr, nullptr);
}

// tail: factors in the tail of the launch -- only when ONE launch takes every layer (all L rows of sq come from
// it); *tail_done says whether that happened.
static int gram_layers_sqnorms(const dpclip_layer* layers, int L, int B, dpclip_dtype dtype, float* sq_layers,
                               int* taken, void* workspace, size_t workspace_bytes, void* stream,
                               const tc::gram::FactorsTail* tail, bool* tail_done) {
    if (tail_done) *tail_done = false;
    if (!layers || L <= 0 || B <= 0 || !sq_layers) return DPCLIP_ERR_INVALID_ARG;
    if (taken) for (int l = 0; l < L; ++l) taken[l] = 0;
    if (dtype != DPCLIP_BF16 || !workspace || workspace_bytes < (size_t)kHeaderBytes) return DPCLIP_OK;
    if (path_switch(SW_NO_GRAM_GROUP)) return DPCLIP_OK;
    namespace g = tc::gram;
    for (int cls = 0; cls < 3; ++cls) {                    // one launch per kernel class (see gram_class)
        GramLayer batch[g::MAX_LAYERS];
        int idx[g::MAX_LAYERS];
        int n = 0;
        auto flush = [&]() -> int {
            // a single layer gains nothing from this entry point: leave it to the per-layer call
            if (n >= 2) {
                const bool with_tail = tail && n == L;             // this launch writes every row of sq
                const int rc = launch_gram_group(batch, n, (int*)workspace, (cudaStream_t)stream, with_tail ? tail : nullptr);
                if (rc) return rc;
                if (taken) for (int i = 0; i < n; ++i) taken[idx[i]] = 1;
                if (with_tail && tail_done) *tail_done = true;
            }
            n = 0;
            return DPCLIP_OK;
        };
        for (int l = 0; l < L; ++l) {
            const dpclip_layer& y = layers[l];
            if (y.T <= 1 || gram_class(y.T) != cls) continue;
            if (check_layer_args(y.A, y.lda, y.Zbar, y.ldz, B, y.T, y.d_in, y.d_out, dtype)) continue;
            if (!tc_eligible(y.A, y.lda, y.Zbar, y.ldz, dtype)) continue;
            int method = y.method;
            if (method == DPCLIP_AUTO) method = dpclip_pick_method(B, y.T, y.d_in, y.d_out, y.lda, y.ldz, dtype);
            if (method != DPCLIP_GRAM) continue;
            batch[n] = {y.A, y.lda, y.Zbar, y.ldz, B, y.T, y.d_in, y.d_out, y.has_bias ? 1 : 0, sq_layers + (size_t)l * B};
            idx[n] = l;
            if (++n == g::MAX_LAYERS) { const int rc = flush(); if (rc) return rc; }
        }
        const int rc = flush();
        if (rc) return rc;
    }
    return DPCLIP_OK;
}

static int shared_clipped_grad_launches(const dpclip_layer* layers, int L, int B, dpclip_dtype dtype,
                                        const float* clip, long clip_ld, float C, float sigma, unsigned long long seed,
                                        unsigned long long stream_id0, int* taken, void* workspace,
                                        size_t workspace_bytes, void* stream);

int dpclip_same_shape_layers_clipped_grad_noise(const dpclip_layer* layers, int L, int B, dpclip_dtype dtype,
                                                const float* clip, float C, float sigma, unsigned long long seed,
                                                unsigned long long stream_id0, int* taken, void* workspace,
                                                size_t workspace_bytes, void* stream) {
    return shared_clipped_grad_launches(layers, L, B, dtype, clip, 0, C, sigma, seed, stream_id0, taken, workspace,
                                        workspace_bytes, stream);
}

// clip_ld = 0: one factor vector for all layers (global clipping); clip_ld > 0: layer l's factors are row l of
// clip[L][clip_ld] (per-layer clipping) -- then only the CTA-pair launches, which take a vector per layer, are made.
static int shared_clipped_grad_launches(const dpclip_layer* layers, int L, int B, dpclip_dtype dtype,
                                        const float* clip, long clip_ld, float C, float sigma, unsigned long long seed,
                                        unsigned long long stream_id0, int* taken, void* workspace,
                                        size_t workspace_bytes, void* stream) {
    if (!layers || L <= 0 || B <= 0) return DPCLIP_ERR_INVALID_ARG;
    if (!(C >= 0.f) || !(sigma >= 0.f)) return DPCLIP_ERR_INVALID_ARG;
    if (taken) for (int l = 0; l < L; ++l) taken[l] = 0;
    if (dtype != DPCLIP_BF16 || !workspace || workspace_bytes < (size_t)kHeaderBytes) return DPCLIP_OK;
    if (path_switch(SW_NO_GRAD_GROUP)) return DPCLIP_OK;
    namespace z = tc::zta;
    constexpr int kMaxTracked = 256;
    if (L > kMaxTracked) return DPCLIP_OK;
    bool done[kMaxTracked] = {false};
    auto candidate = [&](const dpclip_layer& y) {
        if (y.T <= 1 || !y.gW || y.ldg != y.d_in || y.d_in % 4 != 0 || (y.has_bias && !y.gb)) return false;
        if (check_layer_args(y.A, y.lda, y.Zbar, y.ldz, B, y.T, y.d_in, y.d_out, dtype)) return false;
        if (!aligned_to(y.gW, 4) || (y.has_bias && !aligned_to(y.gb, 4))) return false;
        return tc_eligible(y.A, y.lda, y.Zbar, y.ldz, dtype);
    };
    // Layers wide enough for the CTA-pair kernel need not have one shape: all that have one T (hence the same
    // rows B*T) go into one stream-K launch, up to eight at a time.
    for (int l0 = 0; l0 < L; ++l0) {
        if (done[l0] || !candidate(layers[l0]) || !pair_tile_ok(layers[l0].d_out)) continue;
        StreamLayer grp[tc::ztp::MAX_LAYERS];
        int idx[tc::ztp::MAX_LAYERS];
        int n = 0, tiles = 0;
        for (int l = l0; l < L && n < tc::ztp::MAX_LAYERS; ++l) {
            const dpclip_layer& y = layers[l];
            if (done[l] || y.T != layers[l0].T || !pair_tile_ok(y.d_out) || !candidate(y)) continue;
            grp[n] = {y.A, y.lda, y.Zbar, y.ldz, y.d_in, y.d_out, y.gW, y.ldg, y.has_bias ? y.gb : nullptr,
                      stream_id0 + 2ull * l, stream_id0 + 2ull * l + 1, clip ? clip + (size_t)l * clip_ld : nullptr};
            idx[n] = l; ++n;
            tiles += pair_tiles(y.d_in, y.d_out);
        }
        if (n < 2) continue;                       // a single layer takes the same kernel through its own call
        // with less workspace than one segment per tile and pair the launch would run on fewer pairs: leave the
        // layers to their own launches then
        if (workspace_bytes < kHeaderBytes + pair_scratch_bytes(tiles)) continue;
        const NoiseSpec ns = {sigma * C, seed, 0, 0};
        bool noise_done = false;
        const int rc = launch_zta_stream(grp, n, B, layers[l0].T, &ns, &noise_done, workspace, workspace_bytes,
                                         (cudaStream_t)stream);
        if (rc < 0) return rc;
        if (rc > 0) continue;
        if (sigma * C > 0.f && !noise_done) return DPCLIP_ERR_UNSUPPORTED;    // candidate() checked dense rows, d_in % 4
        if (!taken) return DPCLIP_ERR_INVALID_ARG;               // without `taken` the caller cannot know
        for (int i = 0; i < n; ++i) { done[idx[i]] = true; taken[idx[i]] = 1; }
    }
    if (clip_ld > 0) return DPCLIP_OK;
    for (int l0 = 0; l0 < L; ++l0) {
        if (done[l0] || !candidate(layers[l0])) continue;
        const dpclip_layer* grp[z::MAX_LAYERS];
        int idx[z::MAX_LAYERS];
        int n = 0;
        for (int l = l0; l < L && n < z::MAX_LAYERS; ++l) {
            const dpclip_layer& y = layers[l];
            if (done[l] || y.T != layers[l0].T || y.d_in != layers[l0].d_in || y.d_out != layers[l0].d_out) continue;
            if (!candidate(y)) continue;
            grp[n] = &y; idx[n] = l; ++n;
        }
        for (int i = 0; i < n; ++i) done[idx[i]] = true;
        if (n < 2) continue;
        {
            // Sharing a launch pays when a layer alone leaves every CTA a short row slice (pipeline fill and
            // epilogue then weigh heavily); layers that already give long slices keep their own launches,
            // whose one-wave split uses the SMs more evenly (measured on two 512 -> 2048 layers at
            // B*T = 32768: 174 us together on 128 CTAs, 2 x 80 us apart on 144).
            const dpclip_layer& y = layers[l0];
            const int bm = y.d_out > 128 ? 256 : 128;
            const int tiles = ceil_div(y.d_out, bm) * ceil_div(y.d_in, z::BN);
            const long nkb = ceil_div((long)B * y.T, 64L);          // 64-row blocks
            const int ksplit = tiles < kNumSMs ? kNumSMs / tiles : 1;
            if (nkb / ksplit >= 32) continue;
        }
        const int rc = launch_zta_tc_group(grp, idx, n, B, clip, sigma * C, seed, stream_id0, workspace, workspace_bytes,
                                           (cudaStream_t)stream);
        if (rc < 0) return rc;
        if (rc == 0 && taken) for (int i = 0; i < n; ++i) taken[idx[i]] = 1;
        if (rc == 0 && !taken) return DPCLIP_ERR_INVALID_ARG;     // without `taken` the caller cannot know
    }
    return DPCLIP_OK;
}

int dpclip_factors(const float* sq_layers, int L, long ld_sq, int B, float C, float* clip, float* norms,
                   int* n_clipped, void* stream) {
    if (!sq_layers || !clip) return DPCLIP_ERR_INVALID_ARG;
    if (L <= 0 || B <= 0 || ld_sq < B || !(C > 0.f)) return DPCLIP_ERR_INVALID_ARG;
    factors_kernel<<<1, 256, 0, (cudaStream_t)stream>>>(sq_layers, L, ld_sq, B, C, clip, norms, n_clipped);
    return launch_status();
}

int dpclip_clipped_grad(const void* A, long lda, const void* Zbar, long ldz, int B, int T, int d_in,
                        int d_out, dpclip_dtype dtype, const float* clip, float* gW, long ldg, float* gb,
                        void* workspace, size_t workspace_bytes, void* stream) {
    int rc = check_layer_args(A, lda, Zbar, ldz, B, T, d_in, d_out, dtype);
    if (rc) return rc;
    if (!gW || ldg < d_in) return DPCLIP_ERR_INVALID_ARG;
    if (!aligned_to(gW, 4) || (gb && !aligned_to(gb, 4))) return DPCLIP_ERR_MISALIGNED;
    if (!workspace || workspace_bytes < workspace_floor(B, T, d_in, d_out, dtype))
        return DPCLIP_ERR_WORKSPACE;
    return clipped_grad_impl(A, lda, Zbar, ldz, B, T, d_in, d_out, dtype, clip, gW, ldg, gb, workspace,
                             workspace_bytes, nullptr, nullptr, (cudaStream_t)stream);
}

int dpclip_clipped_grad_noise(const void* A, long lda, const void* Zbar, long ldz, int B, int T, int d_in,
                              int d_out, dpclip_dtype dtype, const float* clip, float* gW, float* gb, float sigma,
                              float C, unsigned long long seed, unsigned long long stream_id_w,
                              unsigned long long stream_id_b, void* workspace, size_t workspace_bytes,
                              void* stream) {
    int rc = check_layer_args(A, lda, Zbar, ldz, B, T, d_in, d_out, dtype);
    if (rc) return rc;
    if (!gW || !(sigma >= 0.f) || !(C >= 0.f)) return DPCLIP_ERR_INVALID_ARG;
    if (!aligned_to(gW, 4) || (gb && !aligned_to(gb, 4))) return DPCLIP_ERR_MISALIGNED;
    if (!workspace || workspace_bytes < workspace_floor(B, T, d_in, d_out, dtype))
        return DPCLIP_ERR_WORKSPACE;
    NoiseSpec ns = {sigma * C, seed, stream_id_w, stream_id_b};
    bool noise_done = false;
    rc = clipped_grad_impl(A, lda, Zbar, ldz, B, T, d_in, d_out, dtype, clip, gW, d_in, gb, workspace,
                           workspace_bytes, &ns, &noise_done, (cudaStream_t)stream);
    if (rc || noise_done) return rc;
    rc = dpclip_add_noise(gW, (size_t)d_out * d_in, sigma, C, seed, stream_id_w, stream);
    if (rc || !gb) return rc;
    return dpclip_add_noise(gb, (size_t)d_out, sigma, C, seed, stream_id_b, stream);
}

static int launch_dp_update(bool adam, float* theta, float* m, float* v, const float* gsum, size_t n, float inv_tau,
                            float C, float sigma, unsigned long long seed, unsigned long long stream_id, float lr,
                            float beta1, float beta2, float eps, int step, void* stream) {
    if (n == 0) return DPCLIP_OK;
    if (!theta || !gsum || (adam && (!m || !v))) return DPCLIP_ERR_INVALID_ARG;
    if (!(sigma >= 0.f) || !(C >= 0.f) || !(inv_tau > 0.f)) return DPCLIP_ERR_INVALID_ARG;
    if (adam && (step < 1 || !(beta1 >= 0.f && beta1 < 1.f) || !(beta2 >= 0.f && beta2 < 1.f))) return DPCLIP_ERR_INVALID_ARG;
    if (!aligned_to(theta, 4) || !aligned_to(gsum, 4) || (adam && (!aligned_to(m, 4) || !aligned_to(v, 4))))
        return DPCLIP_ERR_MISALIGNED;
    UpdateParams p;
    memset(&p, 0, sizeof(p));
    p.theta = theta; p.m = m; p.v = v; p.gsum = gsum; p.n = n;
    p.inv_tau = inv_tau; p.scale = sigma * C; p.lr = lr; p.beta1 = beta1; p.beta2 = beta2; p.eps = eps;
    if (adam) {
        p.inv_c1 = (float)(1.0 / (1.0 - pow((double)beta1, (double)step)));
        p.inv_c2 = (float)(1.0 / (1.0 - pow((double)beta2, (double)step)));
    }
    p.k0 = (uint32_t)seed; p.k1 = (uint32_t)(seed >> 32); p.s0 = (uint32_t)stream_id; p.s1 = (uint32_t)(stream_id >> 32);
    p.vec_ok = aligned_to(theta, 16) && aligned_to(gsum, 16) && (!adam || (aligned_to(m, 16) && aligned_to(v, 16)));
    const size_t nq = (n + 3) / 4;
    size_t blocks = (nq + 255) / 256;
    const size_t cap = (size_t)kNumSMs * 16;
    if (blocks > cap) blocks = cap;
    if (adam) dp_update_kernel<true><<<(unsigned)blocks, 256, 0, (cudaStream_t)stream>>>(p);
    else dp_update_kernel<false><<<(unsigned)blocks, 256, 0, (cudaStream_t)stream>>>(p);
    return launch_status();
}

int dpclip_dp_sgd_step(float* theta, const float* gsum, size_t n, float inv_tau, float C, float sigma,
                       unsigned long long seed, unsigned long long stream_id, float lr, void* stream) {
    return launch_dp_update(false, theta, nullptr, nullptr, gsum, n, inv_tau, C, sigma, seed, stream_id, lr, 0.f, 0.f,
                            0.f, 1, stream);
}

int dpclip_dp_adam_step(float* theta, float* m, float* v, const float* gsum, size_t n, float inv_tau, float C,
                        float sigma, unsigned long long seed, unsigned long long stream_id, float lr, float beta1,
                        float beta2, float eps, int step, void* stream) {
    return launch_dp_update(true, theta, m, v, gsum, n, inv_tau, C, sigma, seed, stream_id, lr, beta1, beta2, eps,
                            step, stream);
}

// Convolution layers given by their input feature map (implicit im2col).
static int conv_setup(SimtParams& p, const void* X, const void* Zbar, int z_channel_major, int B, const dpclip_conv* g,
                      int d_out, dpclip_dtype dtype, int has_bias, int* T_out) {
    if (!X || !Zbar || !g) return DPCLIP_ERR_INVALID_ARG;
    if (B <= 0 || d_out <= 0 || g->C <= 0 || g->H <= 0 || g->W <= 0 || g->kh <= 0 || g->kw <= 0 || g->stride <= 0 ||
        g->pad < 0) return DPCLIP_ERR_INVALID_ARG;
    if (dtype != DPCLIP_F32 && dtype != DPCLIP_BF16) return DPCLIP_ERR_INVALID_ARG;
    if (g->H + 2 * g->pad < g->kh || g->W + 2 * g->pad < g->kw) return DPCLIP_ERR_INVALID_ARG;
    if (!aligned_to(X, elt_size(dtype)) || !aligned_to(Zbar, elt_size(dtype))) return DPCLIP_ERR_MISALIGNED;
    const int Ho = (g->H + 2 * g->pad - g->kh) / g->stride + 1, Wo = (g->W + 2 * g->pad - g->kw) / g->stride + 1;
    const long T = (long)Ho * Wo, d_in = (long)g->C * g->kh * g->kw;
    if (T * B > 0x7FFFFFFFL || d_in > 0x7FFFFFFFL || (long)g->C * g->H * g->W > 0x7FFFFFFFL) return DPCLIP_ERR_INVALID_ARG;
    fill_simt_params(p, X, d_in, Zbar, d_out, (int)T, (int)d_in, d_out, has_bias, dtype);
    p.vec_a = 0;
    p.vec_z = z_channel_major ? 0 : vec4_ok(Zbar, d_out, dtype);
    p.cC = g->C; p.cH = g->H; p.cW = g->W; p.kh = g->kh; p.kw = g->kw; p.stride = g->stride; p.pad = g->pad;
    p.Wo = Wo; p.z_cm = z_channel_major ? 1 : 0;
    *T_out = (int)T;
    return DPCLIP_OK;
}

// fp32, dL/dZ as [B][T][d_out] with 16-byte rows, enough work: the tensor-core kernel with the A operand gathered
static bool conv_tf32_ok(const SimtParams& p, const void* X, const void* Zbar, int z_channel_major, int B, int T,
                         dpclip_dtype dtype, const void* workspace, size_t workspace_bytes, tc::ConvGather* cg) {
    if (path_switch(SW_FORCE_SIMT)) return false;
    if (dtype != DPCLIP_F32 || z_channel_major || !workspace || workspace_bytes < (size_t)kHeaderBytes) return false;
    if (!aligned_to(Zbar, 16) || p.d_out % 4 != 0 || p.kh > 255 || p.kw > 255) return false;
    if ((double)B * T * p.d_in * p.d_out < 32.0 * 1024 * 1024) return false;
    cg->X = static_cast<const float*>(X);
    cg->C = p.cC; cg->H = p.cH; cg->W = p.cW; cg->kh = p.kh; cg->kw = p.kw; cg->stride = p.stride; cg->pad = p.pad;
    cg->Wo = p.Wo;
    return true;
}

// bf16 convolution layers on the tensor cores (implicit im2col): see kernels_conv_tc.cuh for the restrictions
static bool conv_tc_ok(const SimtParams& p, const void* X, const void* Zbar, int z_channel_major, int B, int T,
                       dpclip_dtype dtype, const void* workspace, size_t workspace_bytes) {
    if (path_switch(SW_FORCE_SIMT)) return false;
    if (path_switch(SW_NO_CONV_TC)) return false;
    if (dtype != DPCLIP_BF16 || !workspace || workspace_bytes < (size_t)kHeaderBytes) return false;
    if (p.stride != 1 || !(p.Wo == 8 || p.Wo == 16 || p.Wo == 32 || p.Wo == 64) || T % 64 != 0) return false;
    if (p.d_out % 8 != 0 || p.d_out > 128) return false;
    const long x_elems = (long)p.cC * p.cH * p.cW;
    if (x_elems * 2 > tc::ctc::X_BYTES || x_elems % 8 != 0) return false;
    return aligned_to(X, 16) && aligned_to(Zbar, 16);
}

extern "C++" {
template <bool GRAD>
static int launch_conv_tc(const SimtParams& sp, const void* X, const void* Zbar, int B, int T, int has_bias,
                          const float* clip, float* sq, float* gW, long ldg, float* gb, void* workspace,
                          size_t workspace_bytes, cudaStream_t st) {
    namespace c = tc::ctc;
    CUtensorMap mz;
    // dL/dZ as [B][T][d_out]: boxes of 64 rows t x 64 columns; as [B][d_out][T]: one box of d_out rows x 64 t
    if (sp.z_cm ? !make_map_bf16(&mz, Zbar, (long)B * sp.d_out, T, T, c::BK, sp.d_out)
                : !make_map_bf16(&mz, Zbar, (long)B * T, sp.d_out, sp.d_out, 64, c::BK)) return DPCLIP_ERR_CUDA;
    c::Params p;
    memset(&p, 0, sizeof(p));
    p.z_cm = sp.z_cm;
    p.X = static_cast<const __nv_bfloat16*>(X);
    p.B = B; p.C = sp.cC; p.H = sp.cH; p.W = sp.cW; p.kh = sp.kh; p.kw = sp.kw; p.pad = sp.pad;
    p.Wo = sp.Wo; p.Ho = T / sp.Wo;
    p.wo_shift = sp.Wo == 8 ? 3 : sp.Wo == 16 ? 4 : sp.Wo == 32 ? 5 : 6;
    p.T = T; p.d_in = sp.d_in; p.d_out = sp.d_out; p.has_bias = has_bias ? 1 : 0;
    p.tiles_n = ceil_div(sp.d_in + p.has_bias, c::BN);
    p.status = static_cast<int*>(workspace);
    int slices = 1;
    if (GRAD) {
        // one wave: as many slices of examples as there are SMs per block of patch columns
        slices = sm_budget() / p.tiles_n;
        if (slices > B) slices = B;
        if (slices < 1) slices = 1;
        p.ex_per_item = ceil_div(B, slices);
        slices = ceil_div(B, p.ex_per_item);
        p.n_items = slices * p.tiles_n;
        const size_t part_bytes = (size_t)p.n_items * 128 * c::BN * 4;
        if (workspace_bytes < (size_t)kHeaderBytes + part_bytes) return 1;        // the caller takes the fp32-ALU kernel
        p.part = reinterpret_cast<float*>(static_cast<char*>(workspace) + kHeaderBytes);
        p.clip = clip;
    } else {
        p.ex_per_item = 1;
        p.n_items = B * p.tiles_n;
        p.sq = sq;
        if (cudaMemsetAsync(sq, 0, sizeof(float) * (size_t)B, st) != cudaSuccess) return DPCLIP_ERR_CUDA;
    }
    if (!enable_smem(tc::conv_tc_kernel<GRAD>, c::SMEM_BYTES)) return DPCLIP_ERR_CUDA;
    const int grid = p.n_items < sm_budget() ? p.n_items : sm_budget();
    tc::conv_tc_kernel<GRAD><<<grid, c::THREADS, c::SMEM_BYTES, st>>>(mz, p);
    int rc = launch_status();
    if (rc || !GRAD) return rc;
    // fixed-order sum of the slices' tiles; the bias sums are column d_in of the tiles
    tc::zta::Params zp;
    memset(&zp, 0, sizeof(zp));
    zp.part = p.part; zp.tiles_n = p.tiles_n; zp.vec_ok = aligned_to(gW, 16) && ldg % 4 == 0;
    tc::ReduceParams r;
    memset(&r, 0, sizeof(r));
    r.part = p.part; r.n_tiles = p.tiles_n; r.tiles_n = p.tiles_n; r.ksplit = slices; r.BM = 128; r.BN = c::BN;
    r.d_out = sp.d_out; r.d_in = sp.d_in; r.gW = gW; r.ldg = ldg; r.gb = gb; r.vec_ok = zp.vec_ok;
    r.bias_col = 1;
    const long n_vec = (long)sp.d_out * ((sp.d_in + 3) / 4);
    int lanes = 1;
    while (lanes < 8 && lanes * 2 <= slices && n_vec * lanes < 2L * kNumSMs * 256) lanes *= 2;
    r.lanes = lanes;
    long blocks = (n_vec + (256 / lanes) - 1) / (256 / lanes);
    if (blocks > 8L * kNumSMs) blocks = 8L * kNumSMs;
    tc::reduce_partials_kernel<<<(unsigned)blocks, 256, 0, st>>>(r);
    return launch_status();
}
}  // extern "C++"

// fp32 dL/dZ in the channel-major layout [B][d_out][T]: the tf32 tensor-core kernel reads [row][feature]
// tiles, so the tensor is rewritten once per call as [B][T][d_out] behind the partial-tile scratch when the
// workspace has room for it (dpclip_conv_workspace_bytes); otherwise the fp32-ALU kernel reads it in place.
// Returns the pointer to use and clears *channel_major when it did.
static const void* conv_f32_rows_of_channel_major(const SimtParams& p, const void* Zbar, int* channel_major, int B, int T,
                                                  dpclip_dtype dtype, void* workspace, size_t workspace_bytes,
                                                  cudaStream_t st, int* rc) {
    *rc = DPCLIP_OK;
    if (dtype != DPCLIP_F32 || !*channel_major || !workspace || B > 65535) return Zbar;
    if (path_switch(SW_FORCE_SIMT)) return Zbar;
    if (p.d_out % 4 != 0 || p.kh > 255 || p.kw > 255) return Zbar;
    if ((double)B * T * p.d_in * p.d_out < 32.0 * 1024 * 1024) return Zbar;           // stays on the fp32-ALU tiles
    const size_t z_bytes = (size_t)B * T * p.d_out * 4;
    if (workspace_bytes < (size_t)kHeaderBytes + kTcScratchBytes + z_bytes) return Zbar;
    float* rows = reinterpret_cast<float*>(static_cast<char*>(workspace) + kHeaderBytes + kTcScratchBytes);
    const dim3 grid(ceil_div(T, 32), ceil_div(p.d_out, 32), B);
    channel_major_to_rows_kernel<<<grid, 256, 0, st>>>(static_cast<const float*>(Zbar), rows, p.d_out, T);
    if (launch_status()) { *rc = DPCLIP_ERR_CUDA; return Zbar; }
    *channel_major = 0;
    return rows;
}

// fp32 first layers with at most 32 patch columns and 32 outputs: write the patch matrix out behind the scratch
// areas above and hand it to the dense entry points (packed narrow tensor-core kernel).  Needs dL/dZ as rows.
// Returns the patch matrix, or NULL when the layer does not qualify or the workspace has no room.
static const float* conv_f32_narrow_patches(const SimtParams& p, const void* X, const void* z_rows, int z_cm, int B, int T,
                                            dpclip_dtype dtype, int has_bias, void* workspace, size_t workspace_bytes,
                                            cudaStream_t st, int* rc) {
    *rc = DPCLIP_OK;
    if (dtype != DPCLIP_F32 || z_cm || !workspace || p.d_out > 32 || p.d_in + (has_bias ? 1 : 0) > 32) return nullptr;
    if (path_switch(SW_FORCE_SIMT)) return nullptr;
    if (path_switch(SW_NO_CONV_PATCHES)) return nullptr;
    if ((double)B * T * p.d_in * p.d_out < 32.0 * 1024 * 1024) return nullptr;
    if (((long)T * p.d_in * 4) % 16 != 0 || ((long)T * p.d_out * 4) % 16 != 0 || !aligned_to(z_rows, 16)) return nullptr;
    const size_t z_bytes = round_up((size_t)B * T * p.d_out * 4, 256), a_bytes = (size_t)B * T * p.d_in * 4;
    if (workspace_bytes < (size_t)kHeaderBytes + kTcScratchBytes + z_bytes + a_bytes) return nullptr;
    float* patches = reinterpret_cast<float*>(static_cast<char*>(workspace) + kHeaderBytes + kTcScratchBytes + z_bytes);
    const long rows = (long)B * T;
    if (rows > 0x7FFFFFFFL - 64) return nullptr;
    im2col_f32_kernel<<<(unsigned)((rows + 63) / 64), 256, 0, st>>>(static_cast<const float*>(X), patches, (int)rows, T,
                                                                    p.d_in, p.cC, p.cH, p.cW, p.kh, p.kw, p.stride, p.pad,
                                                                    p.Wo);
    if (launch_status()) { *rc = DPCLIP_ERR_CUDA; return nullptr; }
    return patches;
}

size_t dpclip_conv_workspace_bytes(int B, const dpclip_conv* geom, int d_out, dpclip_dtype dtype, int z_channel_major) {
    if (!geom || B <= 0 || d_out <= 0 || geom->stride <= 0) return kHeaderBytes;
    const int Ho = (geom->H + 2 * geom->pad - geom->kh) / geom->stride + 1;
    const int Wo = (geom->W + 2 * geom->pad - geom->kw) / geom->stride + 1;
    if (Ho <= 0 || Wo <= 0) return kHeaderBytes;
    const int T = Ho * Wo;
    size_t w = dpclip_workspace_bytes(B, T, geom->C * geom->kh * geom->kw, d_out, dtype, DPCLIP_AUTO);
    if (dtype == DPCLIP_F32 && w >= (size_t)kHeaderBytes + kTcScratchBytes) {
        const int d_in = geom->C * geom->kh * geom->kw;
        const bool narrow = d_out <= 32 && d_in + 1 <= 32;
        if (z_channel_major || narrow) w += round_up((size_t)B * T * d_out * 4, 256);   // the row-major copy of dL/dZ
        if (narrow) w += (size_t)B * T * d_in * 4;                                       // the patch matrix
    }
    return w;
}

int dpclip_conv_sqnorms(const void* X, const void* Zbar, int z_channel_major, int B, const dpclip_conv* geom,
                        int d_out, dpclip_dtype dtype, int has_bias, float* sq_layer, void* workspace,
                        size_t workspace_bytes, void* stream) {
    SimtParams p;
    int T = 0;
    int rc = conv_setup(p, X, Zbar, z_channel_major, B, geom, d_out, dtype, has_bias, &T);
    if (rc) return rc;
    if (!sq_layer) return DPCLIP_ERR_INVALID_ARG;
    if (B > 65535) return DPCLIP_ERR_UNSUPPORTED;
    cudaStream_t st = (cudaStream_t)stream;
    tc::ConvGather cg;
    if (conv_tc_ok(p, X, Zbar, z_channel_major, B, T, dtype, workspace, workspace_bytes))
        return launch_conv_tc<false>(p, X, Zbar, B, T, has_bias, nullptr, sq_layer, nullptr, 0, nullptr, workspace,
                                     workspace_bytes, st);
    int z_cm = z_channel_major;
    const void* z_rows = conv_f32_rows_of_channel_major(p, Zbar, &z_cm, B, T, dtype, workspace, workspace_bytes, st, &rc);
    if (rc) return rc;
    if (const float* patches = conv_f32_narrow_patches(p, X, z_rows, z_cm, B, T, dtype, has_bias, workspace, workspace_bytes,
                                                       st, &rc))
        return dpclip_layer_sqnorms(patches, p.d_in, z_rows, d_out, B, T, p.d_in, d_out, dtype, has_bias, DPCLIP_AUTO,
                                    sq_layer, workspace, (size_t)kHeaderBytes + kTcScratchBytes, stream);
    if (rc) return rc;
    if (conv_tf32_ok(p, X, z_rows, z_cm, B, T, dtype, workspace, workspace_bytes, &cg))
        return launch_zta_tf32(nullptr, p.d_in, z_rows, d_out, B, T, p.d_in, d_out, true, has_bias, nullptr, nullptr, 0,
                               nullptr, sq_layer, workspace, workspace_bytes, nullptr, nullptr, st, &cg);
    const int n_tiles = p.tiles_m * p.tiles_n;
    int split = ceil_div(2 * kNumSMs, B);
    if (split > n_tiles) split = n_tiles;
    if (split < 1) split = 1;
    p.sq = sq_layer;
    p.use_atomic = split > 1;
    if (p.use_atomic && cudaMemsetAsync(sq_layer, 0, sizeof(float) * (size_t)B, st) != cudaSuccess) return DPCLIP_ERR_CUDA;
    dim3 grid(split, B);
    if (dtype == DPCLIP_F32) zta_simt_kernel<float, false, true><<<grid, SIMT_THREADS, 0, st>>>(p);
    else zta_simt_kernel<__nv_bfloat16, false, true><<<grid, SIMT_THREADS, 0, st>>>(p);
    return launch_status();
}

int dpclip_conv_clipped_grad(const void* X, const void* Zbar, int z_channel_major, int B, const dpclip_conv* geom,
                             int d_out, dpclip_dtype dtype, const float* clip, float* gW, long ldg, float* gb,
                             void* workspace, size_t workspace_bytes, void* stream) {
    SimtParams p;
    int T = 0;
    int rc = conv_setup(p, X, Zbar, z_channel_major, B, geom, d_out, dtype, gb != nullptr, &T);
    if (rc) return rc;
    if (!gW || ldg < p.d_in) return DPCLIP_ERR_INVALID_ARG;
    if (!aligned_to(gW, 4) || (gb && !aligned_to(gb, 4))) return DPCLIP_ERR_MISALIGNED;
    cudaStream_t st = (cudaStream_t)stream;
    tc::ConvGather cg;
    if (conv_tc_ok(p, X, Zbar, z_channel_major, B, T, dtype, workspace, workspace_bytes)) {
        rc = launch_conv_tc<true>(p, X, Zbar, B, T, gb != nullptr, clip, nullptr, gW, ldg, gb, workspace, workspace_bytes, st);
        if (rc <= 0) return rc;
    }
    int z_cm = z_channel_major;
    const void* z_rows = conv_f32_rows_of_channel_major(p, Zbar, &z_cm, B, T, dtype, workspace, workspace_bytes, st, &rc);
    if (rc) return rc;
    if (const float* patches = conv_f32_narrow_patches(p, X, z_rows, z_cm, B, T, dtype, gb != nullptr, workspace,
                                                       workspace_bytes, st, &rc))
        return dpclip_clipped_grad(patches, p.d_in, z_rows, d_out, B, T, p.d_in, d_out, dtype, clip, gW, ldg, gb, workspace,
                                   (size_t)kHeaderBytes + kTcScratchBytes, stream);
    if (rc) return rc;
    if (conv_tf32_ok(p, X, z_rows, z_cm, B, T, dtype, workspace, workspace_bytes, &cg) &&
        workspace_bytes >= (size_t)kHeaderBytes + kTcScratchBytes)
        return launch_zta_tf32(nullptr, p.d_in, z_rows, d_out, B, T, p.d_in, d_out, false, 0, clip, gW, ldg, gb, nullptr,
                               workspace, workspace_bytes, nullptr, nullptr, st, &cg);
    const int n_tiles = p.tiles_m * p.tiles_n;
    const long rows = (long)B * T;
    long ksplit = ceil_div(4 * kNumSMs, n_tiles);
    const long max_split = (rows + 4 * SIMT_BK - 1) / (4 * SIMT_BK);
    if (ksplit > max_split) ksplit = max_split;
    if (ksplit < 1) ksplit = 1;
    if (ksplit > 65535) ksplit = 65535;
    long per = (rows + ksplit - 1) / ksplit;
    per = (per + SIMT_BK - 1) / SIMT_BK * SIMT_BK;
    ksplit = (rows + per - 1) / per;
    p.clip = clip; p.gW = gW; p.ldg = ldg; p.gb = gb;
    p.rows_total = rows; p.rows_per_split = per;
    p.use_atomic = ksplit > 1;
    if (p.use_atomic) {
        if (cudaMemset2DAsync(gW, sizeof(float) * (size_t)ldg, 0, sizeof(float) * (size_t)p.d_in, d_out, st) != cudaSuccess)
            return DPCLIP_ERR_CUDA;
        if (gb && cudaMemsetAsync(gb, 0, sizeof(float) * (size_t)d_out, st) != cudaSuccess) return DPCLIP_ERR_CUDA;
    }
    dim3 grid(n_tiles, (unsigned)ksplit);
    if (dtype == DPCLIP_F32) zta_simt_kernel<float, true, true><<<grid, SIMT_THREADS, 0, st>>>(p);
    else zta_simt_kernel<__nv_bfloat16, true, true><<<grid, SIMT_THREADS, 0, st>>>(p);
    return launch_status();
}

int dpclip_step_noise(const dpclip_layer* layers, int L, float C, float sigma, unsigned long long seed,
                      unsigned long long stream_id0, void* stream) {
    if (!layers || L <= 0 || !(C >= 0.f) || !(sigma >= 0.f)) return DPCLIP_ERR_INVALID_ARG;
    if (sigma * C == 0.f) return DPCLIP_OK;
    cudaStream_t st = (cudaStream_t)stream;
    for (int l0 = 0; l0 < L; l0 += NOISE_BATCH_MAX / 2) {          // at most 64 layers (128 tensors) per launch
        NoiseBatchParams p;
        memset(&p, 0, sizeof(p));
        p.scale = sigma * C; p.k0 = (uint32_t)seed; p.k1 = (uint32_t)(seed >> 32);
        int blocks = 0;
        const int l1 = l0 + NOISE_BATCH_MAX / 2 < L ? l0 + NOISE_BATCH_MAX / 2 : L;
        for (int l = l0; l < l1; ++l) {
            const dpclip_layer& y = layers[l];
            if (!y.gW || y.d_in <= 0 || y.d_out <= 0) return DPCLIP_ERR_INVALID_ARG;
            if (y.ldg != y.d_in) return DPCLIP_ERR_UNSUPPORTED;      // noise indexes the dense tensor
            if (y.has_bias && !y.gb) return DPCLIP_ERR_INVALID_ARG;
            if (!aligned_to(y.gW, 4) || (y.gb && !aligned_to(y.gb, 4))) return DPCLIP_ERR_MISALIGNED;
            auto add = [&](float* g, size_t n, unsigned long long sid) {
                const size_t nq = (n + 3) / 4;
                size_t b = (nq + 255) / 256;
                if (b > (size_t)kNumSMs * 4) b = (size_t)kNumSMs * 4;
                p.g[p.count] = g; p.n[p.count] = n; p.sid[p.count] = sid; p.blk_begin[p.count] = blocks;
                blocks += (int)b; ++p.count;
            };
            add(y.gW, (size_t)y.d_out * y.d_in, stream_id0 + 2ull * l);
            if (y.has_bias) add(y.gb, (size_t)y.d_out, stream_id0 + 2ull * l + 1);
        }
        p.blk_begin[p.count] = blocks;
        noise_batch_kernel<<<blocks, 256, 0, st>>>(p);
        if (launch_status()) return DPCLIP_ERR_CUDA;
    }
    return DPCLIP_OK;
}

int dpclip_t1_layers_supported(const dpclip_layer* layers, int L, int B, dpclip_dtype dtype) {
    if (!layers || L <= 0 || B <= 0) return 0;
    T1Group g;
    if (prepare_t1_group(g, layers, L, B, dtype, 1.f, 0.f, 0, 0, nullptr, nullptr, /*mixed_only=*/false)) return 0;
    return g.active ? 1 : 0;
}

int dpclip_t1_layers_sqnorms(const dpclip_layer* layers, int L, int B, dpclip_dtype dtype, float* sq_layers,
                             void* stream) {
    if (!layers || L <= 0 || B <= 0 || !sq_layers) return DPCLIP_ERR_INVALID_ARG;
    T1Group g;
    int rc = prepare_t1_group(g, layers, L, B, dtype, 1.f, 0.f, 0, 0, sq_layers, nullptr, /*mixed_only=*/false);
    if (rc) return rc;
    if (!g.active) return DPCLIP_ERR_UNSUPPORTED;
    if (dtype == DPCLIP_F32) t1_all_norms_kernel<float><<<g.p.L * B, 128, 0, (cudaStream_t)stream>>>(g.p);
    else t1_all_norms_kernel<__nv_bfloat16><<<g.p.L * B, 128, 0, (cudaStream_t)stream>>>(g.p);
    return launch_status();
}

int dpclip_t1_layers_clipped_grad_noise(const dpclip_layer* layers, int L, int B, dpclip_dtype dtype,
                                        const float* clip, float C, float sigma, unsigned long long seed,
                                        unsigned long long stream_id0, void* workspace, size_t workspace_bytes,
                                        void* stream) {
    if (!layers || L <= 0 || B <= 0 || !clip) return DPCLIP_ERR_INVALID_ARG;
    if (!(C > 0.f) || !(sigma >= 0.f)) return DPCLIP_ERR_INVALID_ARG;
    if (!workspace || workspace_bytes < (size_t)kHeaderBytes) return DPCLIP_ERR_WORKSPACE;
    T1Group g;
    int rc = prepare_t1_group(g, layers, L, B, dtype, C, sigma, seed, stream_id0, nullptr, clip, /*mixed_only=*/false);
    if (rc) return rc;
    if (!g.active) return DPCLIP_ERR_UNSUPPORTED;
    rc = launch_fused_t1_tf32(g.p, false, dtype, workspace, workspace_bytes, (cudaStream_t)stream);
    return rc > 0 ? DPCLIP_ERR_UNSUPPORTED : rc;
}

int dpclip_elementwise_sqnorms(const void* Hbar, long ldh, const void* Zbar, long ldz, int B, int T, int d,
                               dpclip_dtype dtype, int has_shift, float* sq_layer, void* stream) {
    int rc = check_layer_args(Hbar, ldh, Zbar, ldz, B, T, d, d, dtype);
    if (rc) return rc;
    if (!sq_layer) return DPCLIP_ERR_INVALID_ARG;
    if (B > 65535) return DPCLIP_ERR_UNSUPPORTED;
    cudaStream_t st = (cudaStream_t)stream;
    const bool vec = vec4_ok(Hbar, ldh, dtype) && vec4_ok(Zbar, ldz, dtype) && d % 4 == 0;
    const int v = vec ? 4 : 1;
    const int cg = (long)ceil_div(d, 64 * v) * B >= 4L * kNumSMs ? 64 : 32;
    const dim3 grid(ceil_div(d, cg * v), B);
    const int use_atomic = grid.x > 1;
    if (use_atomic && cudaMemsetAsync(sq_layer, 0, sizeof(float) * (size_t)B, st) != cudaSuccess) return DPCLIP_ERR_CUDA;
    if (dtype == DPCLIP_F32) launch_ew_norm<float>(vec, cg, grid, st, Hbar, ldh, Zbar, ldz, T, d, has_shift, sq_layer, use_atomic);
    else launch_ew_norm<__nv_bfloat16>(vec, cg, grid, st, Hbar, ldh, Zbar, ldz, T, d, has_shift, sq_layer, use_atomic);
    return launch_status();
}

int dpclip_elementwise_clipped_grad(const void* Hbar, long ldh, const void* Zbar, long ldz, int B, int T, int d,
                                    dpclip_dtype dtype, const float* clip, float* g_scale, float* g_shift,
                                    void* stream) {
    int rc = check_layer_args(Hbar, ldh, Zbar, ldz, B, T, d, d, dtype);
    if (rc) return rc;
    if (!g_scale) return DPCLIP_ERR_INVALID_ARG;
    if (!aligned_to(g_scale, 4) || (g_shift && !aligned_to(g_shift, 4))) return DPCLIP_ERR_MISALIGNED;
    cudaStream_t st = (cudaStream_t)stream;
    const bool vec = vec4_ok(Hbar, ldh, dtype) && vec4_ok(Zbar, ldz, dtype) && d % 4 == 0;
    const int v = vec ? 4 : 1;
    const long R = (long)B * T;
    const int cg = 64;
    const int col_blocks = ceil_div(d, cg * v);
    // about eight CTAs per SM in all (measured: 190 vs 217 us with four on 1 GB of bf16 input), and at least
    // 256 rows per CTA: every CTA ends with one atomic per column, and with 64-row CTAs those adds (512 per
    // address at B*T = 32768, d = 512) cost more than the rows (38.9 vs 26.6 us)
    long slices = (8L * kNumSMs + col_blocks - 1) / col_blocks;
    if (slices > (R + 255) / 256) slices = (R + 255) / 256;
    if (slices < 1) slices = 1;
    if (slices > 65535) slices = 65535;
    const long rows_per_cta = (R + slices - 1) / slices;
    const dim3 grid(col_blocks, (unsigned)ceil_div(R, rows_per_cta));
    if (cudaMemsetAsync(g_scale, 0, sizeof(float) * (size_t)d, st) != cudaSuccess) return DPCLIP_ERR_CUDA;
    if (g_shift && cudaMemsetAsync(g_shift, 0, sizeof(float) * (size_t)d, st) != cudaSuccess) return DPCLIP_ERR_CUDA;
    if (dtype == DPCLIP_F32) launch_ew_grad<float>(vec, cg, grid, st, Hbar, ldh, Zbar, ldz, R, rows_per_cta, T, d, clip, g_scale, g_shift);
    else launch_ew_grad<__nv_bfloat16>(vec, cg, grid, st, Hbar, ldh, Zbar, ldz, R, rows_per_cta, T, d, clip, g_scale, g_shift);
    return launch_status();
}

int dpclip_add_noise(float* g, size_t n, float sigma, float C, unsigned long long seed,
                     unsigned long long stream_id, void* stream) {
    if (n == 0) return DPCLIP_OK;
    if (!g || !(sigma >= 0.f) || !(C >= 0.f)) return DPCLIP_ERR_INVALID_ARG;
    if (!aligned_to(g, 4)) return DPCLIP_ERR_MISALIGNED;
    if (sigma * C == 0.f) return DPCLIP_OK;          // nothing to add: no launch
    const size_t nq = (n + 3) / 4;
    size_t blocks = (nq + 255) / 256;
    const size_t cap = (size_t)kNumSMs * 16;
    if (blocks > cap) blocks = cap;
    noise_kernel<<<(unsigned)blocks, 256, 0, (cudaStream_t)stream>>>(
        g, n, sigma * C, (uint32_t)seed, (uint32_t)(seed >> 32), (uint32_t)stream_id,
        (uint32_t)(stream_id >> 32), aligned_to(g, 16) ? 1 : 0);
    return launch_status();
}

// Norms / clipped sum + noise of a layer that is not a dense product (element-wise parameters, convolution
// given by its feature map): the per-layer entry points, with the layer's row of sq and its noise streams.
static int other_kind_sqnorms(const dpclip_model_layer& m, int B, dpclip_dtype dtype, float* sq_row, void* workspace,
                              size_t workspace_bytes, void* stream) {
    const dpclip_layer& y = m.layer;
    if (m.kind == DPCLIP_KIND_ELEMENTWISE) {
        if (y.d_in != y.d_out) return DPCLIP_ERR_INVALID_ARG;
        return dpclip_elementwise_sqnorms(y.A, y.lda, y.Zbar, y.ldz, B, y.T, y.d_in, dtype, y.has_bias, sq_row, stream);
    }
    if (m.kind == DPCLIP_KIND_CONV)
        return dpclip_conv_sqnorms(y.A, y.Zbar, m.z_channel_major, B, &m.conv, y.d_out, dtype, y.has_bias, sq_row,
                                   workspace, workspace_bytes, stream);
    return DPCLIP_ERR_INVALID_ARG;
}

static int other_kind_clipped_grad_noise(const dpclip_model_layer& m, int B, dpclip_dtype dtype, const float* clip,
                                         float C, float sigma, unsigned long long seed, unsigned long long sid_w,
                                         unsigned long long sid_b, void* workspace, size_t workspace_bytes,
                                         void* stream) {
    const dpclip_layer& y = m.layer;
    float* gb = y.has_bias ? y.gb : nullptr;
    if (!y.gW || (y.has_bias && !gb)) return DPCLIP_ERR_INVALID_ARG;
    size_t n_w = 0;
    int rc;
    if (m.kind == DPCLIP_KIND_ELEMENTWISE) {
        if (y.d_in != y.d_out) return DPCLIP_ERR_INVALID_ARG;
        rc = dpclip_elementwise_clipped_grad(y.A, y.lda, y.Zbar, y.ldz, B, y.T, y.d_in, dtype, clip, y.gW, gb, stream);
        n_w = (size_t)y.d_in;
    } else if (m.kind == DPCLIP_KIND_CONV) {
        const long d_in = (long)m.conv.C * m.conv.kh * m.conv.kw;
        if (y.ldg != d_in) return DPCLIP_ERR_UNSUPPORTED;        // noise indexes the dense tensor
        rc = dpclip_conv_clipped_grad(y.A, y.Zbar, m.z_channel_major, B, &m.conv, y.d_out, dtype, clip, y.gW, y.ldg, gb,
                                      workspace, workspace_bytes, stream);
        n_w = (size_t)y.d_out * (size_t)d_in;
    } else {
        return DPCLIP_ERR_INVALID_ARG;
    }
    if (rc) return rc;
    rc = dpclip_add_noise(y.gW, n_w, sigma, C, seed, sid_w, stream);
    if (rc) return rc;
    if (gb) rc = dpclip_add_noise(gb, m.kind == DPCLIP_KIND_ELEMENTWISE ? (size_t)y.d_in : (size_t)y.d_out, sigma, C,
                                  seed, sid_b, stream);
    return rc;
}

// The streams a step may spread its layers over.  Lane 0 is the caller's stream: the step starts and ends
// there.  fork() makes every other lane wait for what lane 0 has enqueued so far, join() makes lane 0 wait for
// what the other lanes have enqueued; both are event record/wait pairs, which a stream capture records as
// graph dependencies.  Every lane has a workspace of its own (launches on different lanes may overlap).
struct Lanes {
    static constexpr int kMax = 8;
    int n = 1;
    cudaStream_t st[kMax] = {};
    void* ws[kMax] = {};
    size_t ws_bytes = 0;
    cudaEvent_t ev[2 * kMax + 2] = {};
    int n_ev = 0;
    ~Lanes() { for (int i = 0; i < n_ev; ++i) cudaEventDestroy(ev[i]); }     // pending work keeps what it needs
    // events are reused between the fork and the join of a stage: a record replaces the earlier one for later waits only
    int event(cudaEvent_t* out) {
        if (n_ev == 2 * kMax + 2) return DPCLIP_ERR_CUDA;
        if (cudaEventCreateWithFlags(&ev[n_ev], cudaEventDisableTiming) != cudaSuccess) return DPCLIP_ERR_CUDA;
        *out = ev[n_ev++];
        return DPCLIP_OK;
    }
    int fork() {
        if (n == 1) return DPCLIP_OK;
        cudaEvent_t e;
        if (event(&e)) return DPCLIP_ERR_CUDA;
        if (cudaEventRecord(e, st[0]) != cudaSuccess) return DPCLIP_ERR_CUDA;
        for (int i = 1; i < n; ++i)
            if (cudaStreamWaitEvent(st[i], e, 0) != cudaSuccess) return DPCLIP_ERR_CUDA;
        return DPCLIP_OK;
    }
    int join() {
        for (int i = 1; i < n; ++i) {
            cudaEvent_t e;
            if (event(&e)) return DPCLIP_ERR_CUDA;
            if (cudaEventRecord(e, st[i]) != cudaSuccess || cudaStreamWaitEvent(st[0], e, 0) != cudaSuccess)
                return DPCLIP_ERR_CUDA;
        }
        return DPCLIP_OK;
    }
};

// The path layer by layer (with the launches that several layers share), Algorithm 1's order: every layer's
// norms, then the factors, then every layer's clipped sum with its noise.  Layers are independent within the
// norm stage and within the clipped-sum stage, so with several lanes the launches of a stage are dealt to the
// lanes (a layer's kernel then starts on SMs the previous layer's kernel has already left): the shared Gram
// launch and the shared same-shape launch on lane 0, the T = 1 group on the last lane, the rest round-robin.
// `other`, when given, is the model's own descriptor array: entries of a kind other than dense have a
// placeholder with T = 0 in `layers`, which every grouping rule below passes over, and go through the two
// functions above.
static int step_general(const dpclip_layer* layers, const dpclip_model_layer* other, int L, int B, dpclip_dtype dtype,
                        float C, float sigma, unsigned long long seed, unsigned long long stream_id0,
                        float* sq_layers, float* clip, float* norms, Lanes& lanes) {
    int rc;
    const int last = lanes.n - 1;
    void* const ws0 = lanes.ws[0];
    const size_t workspace_bytes = lanes.ws_bytes;
    T1Group t1;
    rc = prepare_t1_group(t1, layers, L, B, dtype, C, sigma, seed, stream_id0, sq_layers, clip);
    if (rc) return rc;
    if (t1.active && (!lanes.ws[last] || workspace_bytes < (size_t)kHeaderBytes)) t1.active = false;
    if ((rc = lanes.fork())) return rc;
    if (t1.active) {
        if (dtype == DPCLIP_F32) t1_all_norms_kernel<float><<<t1.p.L * B, 128, 0, lanes.st[last]>>>(t1.p);
        else t1_all_norms_kernel<__nv_bfloat16><<<t1.p.L * B, 128, 0, lanes.st[last]>>>(t1.p);
        if (launch_status()) return DPCLIP_ERR_CUDA;
    }
    int in_gram_group[64];
    const bool track = L <= 64;
    bool any_gram = false;
    bool factors_done = false;
    if (track) {
        // when one Gram launch takes every layer of the model, its last CTA also computes the factors
        const tc::gram::FactorsTail tail = {sq_layers, L, (long)B, B, C, clip, norms, nullptr};
        rc = gram_layers_sqnorms(layers, L, B, dtype, sq_layers, in_gram_group, ws0, workspace_bytes, lanes.st[0],
                                 (!t1.active && !other && !path_switch(SW_NO_FACTORS_TAIL)) ? &tail : nullptr, &factors_done);
        if (rc) return rc;
        for (int l = 0; l < L; ++l) any_gram = any_gram || in_gram_group[l];
    }
    // SM shares for the per-layer launches of a stage (see t_sm_budget): only when several of them run side by
    // side on different lanes, no launch shared by several layers is in the stage, and the stage is small
    const size_t es = elt_size(dtype);
    auto layer_bytes = [&](int l) -> double {
        if (other && other[l].kind == DPCLIP_KIND_CONV) {
            const dpclip_conv& g = other[l].conv;
            const double Ho = (g.H + 2 * g.pad - g.kh) / g.stride + 1, Wo = (g.W + 2 * g.pad - g.kw) / g.stride + 1;
            return (double)B * ((double)g.C * g.H * g.W + Ho * Wo * other[l].layer.d_out) * es;
        }
        const dpclip_layer& y = other && other[l].kind != DPCLIP_KIND_DENSE ? other[l].layer : layers[l];
        return (double)B * y.T * ((double)y.d_in + y.d_out) * es;
    };
    auto stage_budgets = [&](const int* skip, bool shared_launch, int* budget) {
        int n_ent = 0;
        double total = 0.0;
        for (int l = 0; l < L; ++l) {
            budget[l] = 0;
            const bool is_other = other && other[l].kind != DPCLIP_KIND_DENSE;
            if (!is_other && ((t1.active && layers[l].T == 1) || (skip && skip[l]))) continue;
            ++n_ent; total += layer_bytes(l);
        }
        // bf16 only: the fp32 forms (three tf32 MMAs per product, four operand planes to prepare, gathers) are
        // bound by their own work, and a share of the SMs stretches them in proportion (measured: the feature-map
        // CNN in fp32 242 -> 312 us with shares, in bf16 98 -> 86 us; the patch-matrix CNN in bf16 94 -> 79 us)
        if (dtype != DPCLIP_BF16 || lanes.n < 2 || n_ent < 2 || shared_launch || total > 400e6 ||
            path_switch(SW_NO_SM_BUDGET)) return;
        const double widen = n_ent > lanes.n ? (double)n_ent / lanes.n : 1.0;      // more launches than lanes: some queue
        for (int l = 0; l < L; ++l) {
            const bool is_other = other && other[l].kind != DPCLIP_KIND_DENSE;
            if (!is_other && ((t1.active && layers[l].T == 1) || (skip && skip[l]))) continue;
            int b = (int)(kNumSMs * layer_bytes(l) / total * widen + 0.5);
            budget[l] = b < 16 ? 16 : (b > kNumSMs ? kNumSMs : b);
        }
    };
    int budget[64] = {0};
    if (track) stage_budgets(in_gram_group, any_gram, budget);
    int k = any_gram ? 1 : 0;                              // lane 0 already carries the shared Gram launch
    for (int l = 0; l < L; ++l) {
        const dpclip_layer& y = layers[l];
        const bool is_other = other && other[l].kind != DPCLIP_KIND_DENSE;
        if (!is_other && ((t1.active && y.T == 1) || (track && in_gram_group[l]))) continue;
        const SmBudgetScope share(track ? budget[l] : 0);
        const int b = k++ % lanes.n;
        if (is_other)
            rc = other_kind_sqnorms(other[l], B, dtype, sq_layers + (size_t)l * B, lanes.ws[b], workspace_bytes, lanes.st[b]);
        else
            rc = dpclip_layer_sqnorms(y.A, y.lda, y.Zbar, y.ldz, B, y.T, y.d_in, y.d_out, dtype, y.has_bias,
                                      (dpclip_method)y.method, sq_layers + (size_t)l * B, lanes.ws[b],
                                      workspace_bytes, lanes.st[b]);
        if (rc) return rc;
    }
    if ((rc = lanes.join())) return rc;
    if (!factors_done) {
        rc = dpclip_factors(sq_layers, L, B, B, C, clip, norms, nullptr, lanes.st[0]);
        if (rc) return rc;
    }
    if ((rc = lanes.fork())) return rc;
    if (t1.active) {
        rc = launch_fused_t1_tf32(t1.p, false, dtype, lanes.ws[last], workspace_bytes, lanes.st[last]);
        if (rc < 0) return rc;
        if (rc > 0) return DPCLIP_ERR_UNSUPPORTED;           // prepare_t1_group checked the same conditions
    }
    int in_grad_group[64];
    bool any_group = false;
    if (track) {
        // the factors came from the tail of the Gram launch, the last kernel of this stream: the first clipped-sum
        // launch may start loading while that tail runs
        const OverlapPrevScope overlap(factors_done);
        rc = dpclip_same_shape_layers_clipped_grad_noise(layers, L, B, dtype, clip, C, sigma, seed, stream_id0,
                                                         in_grad_group, ws0, workspace_bytes, lanes.st[0]);
        if (rc) return rc;
        for (int l = 0; l < L; ++l) any_group = any_group || in_grad_group[l];
    }
    if (track) stage_budgets(in_grad_group, any_group, budget);
    k = any_group ? 1 : 0;
    for (int l = 0; l < L; ++l) {
        const dpclip_layer& y = layers[l];
        const bool is_other = other && other[l].kind != DPCLIP_KIND_DENSE;
        if (!is_other && ((t1.active && y.T == 1) || (track && in_grad_group[l]))) continue;
        const SmBudgetScope share(track ? budget[l] : 0);
        const int b = k++ % lanes.n;
        void* const stream = lanes.st[b];
        void* const workspace = lanes.ws[b];
        if (is_other) {
            rc = other_kind_clipped_grad_noise(other[l], B, dtype, clip, C, sigma, seed, stream_id0 + 2ull * l,
                                               stream_id0 + 2ull * l + 1, workspace, workspace_bytes, stream);
            if (rc) return rc;
            continue;
        }
        float* gb = y.has_bias ? y.gb : nullptr;
        if (y.has_bias && !gb) return DPCLIP_ERR_INVALID_ARG;
        // noise indexes the dense d_out x d_in tensor, so the step wants unpadded output rows
        if (y.ldg != y.d_in) return DPCLIP_ERR_UNSUPPORTED;
        rc = check_layer_args(y.A, y.lda, y.Zbar, y.ldz, B, y.T, y.d_in, y.d_out, dtype);
        if (rc) return rc;
        if (!y.gW) return DPCLIP_ERR_INVALID_ARG;
        NoiseSpec ns = {sigma * C, seed, stream_id0 + 2ull * l, stream_id0 + 2ull * l + 1};
        bool noise_done = false;
        rc = clipped_grad_impl(y.A, y.lda, y.Zbar, y.ldz, B, y.T, y.d_in, y.d_out, dtype, clip, y.gW, y.ldg, gb,
                               workspace, workspace_bytes, &ns, &noise_done, (cudaStream_t)stream);
        if (rc) return rc;
        if (!noise_done) {
            rc = dpclip_add_noise(y.gW, (size_t)y.d_out * y.d_in, sigma, C, seed, ns.sid_w, stream);
            if (rc) return rc;
            if (gb) {
                rc = dpclip_add_noise(gb, (size_t)y.d_out, sigma, C, seed, ns.sid_b, stream);
                if (rc) return rc;
            }
        }
    }
    return lanes.join();
}

// Lanes of a one-stream call, and of a several-streams call (argument checks included).
static void one_lane(Lanes& lanes, void* workspace, size_t workspace_bytes, void* stream) {
    lanes.n = 1; lanes.st[0] = (cudaStream_t)stream; lanes.ws[0] = workspace; lanes.ws_bytes = workspace_bytes;
}
static int many_lanes(Lanes& lanes, int n_streams, void* const* streams, void* const* workspaces, size_t workspace_bytes) {
    if (n_streams < 1 || n_streams > Lanes::kMax || !streams || !workspaces) return DPCLIP_ERR_INVALID_ARG;
    lanes.n = n_streams; lanes.ws_bytes = workspace_bytes;
    for (int i = 0; i < n_streams; ++i) {
        lanes.st[i] = (cudaStream_t)streams[i]; lanes.ws[i] = workspaces[i];
        for (int j = 0; j < i; ++j)
            if (streams[i] == streams[j] || (workspaces[i] && workspaces[i] == workspaces[j])) return DPCLIP_ERR_INVALID_ARG;
    }
    return DPCLIP_OK;
}

static int step_args_ok(const void* layers, int L, int B, dpclip_dtype dtype, float C, float sigma, const float* sq_layers,
                        const float* clip) {
    if (!layers || L <= 0 || B <= 0 || !sq_layers || !clip) return DPCLIP_ERR_INVALID_ARG;
    if (!(C > 0.f) || !(sigma >= 0.f)) return DPCLIP_ERR_INVALID_ARG;
    if (dtype != DPCLIP_F32 && dtype != DPCLIP_BF16) return DPCLIP_ERR_INVALID_ARG;
    return DPCLIP_OK;
}

static int step_dense(const dpclip_layer* layers, int L, int B, dpclip_dtype dtype, float C, float sigma,
                      unsigned long long seed, unsigned long long stream_id0, float* sq_layers, float* clip,
                      float* norms, Lanes& lanes) {
    const int rc = try_fused_t1_step(layers, L, B, dtype, C, sigma, seed, stream_id0, sq_layers, clip, norms, lanes.ws[0],
                                     lanes.ws_bytes, lanes.st[0]);
    if (rc <= 0) return rc;                  // done (0) or argument error (< 0); 1 = take the general path
    return step_general(layers, nullptr, L, B, dtype, C, sigma, seed, stream_id0, sq_layers, clip, norms, lanes);
}

static int step_model(const dpclip_model_layer* layers, int L, int B, dpclip_dtype dtype, float C, float sigma,
                      unsigned long long seed, unsigned long long stream_id0, float* sq_layers, float* clip,
                      float* norms, Lanes& lanes) {
    constexpr int kMaxLayers = 256;
    if (L > kMaxLayers) return DPCLIP_ERR_INVALID_ARG;
    dpclip_layer dense[kMaxLayers];
    bool all_dense = true;
    for (int l = 0; l < L; ++l) {
        if (layers[l].kind == DPCLIP_KIND_DENSE) { dense[l] = layers[l].layer; continue; }
        if (layers[l].kind != DPCLIP_KIND_ELEMENTWISE && layers[l].kind != DPCLIP_KIND_CONV) return DPCLIP_ERR_INVALID_ARG;
        memset(&dense[l], 0, sizeof(dense[l]));             // T = 0: no grouping rule takes it
        all_dense = false;
    }
    if (all_dense) return step_dense(dense, L, B, dtype, C, sigma, seed, stream_id0, sq_layers, clip, norms, lanes);
    return step_general(dense, layers, L, B, dtype, C, sigma, seed, stream_id0, sq_layers, clip, norms, lanes);
}

int dpclip_step(const dpclip_layer* layers, int L, int B, dpclip_dtype dtype, float C, float sigma,
                unsigned long long seed, unsigned long long stream_id0, float* sq_layers, float* clip,
                float* norms, void* workspace, size_t workspace_bytes, void* stream) {
    int rc = step_args_ok(layers, L, B, dtype, C, sigma, sq_layers, clip);
    if (rc) return rc;
    Lanes lanes;
    one_lane(lanes, workspace, workspace_bytes, stream);
    return step_dense(layers, L, B, dtype, C, sigma, seed, stream_id0, sq_layers, clip, norms, lanes);
}

int dpclip_step_streams(const dpclip_layer* layers, int L, int B, dpclip_dtype dtype, float C, float sigma,
                        unsigned long long seed, unsigned long long stream_id0, float* sq_layers, float* clip,
                        float* norms, int n_streams, void* const* streams, void* const* workspaces,
                        size_t workspace_bytes) {
    int rc = step_args_ok(layers, L, B, dtype, C, sigma, sq_layers, clip);
    if (rc) return rc;
    Lanes lanes;
    if ((rc = many_lanes(lanes, n_streams, streams, workspaces, workspace_bytes))) return rc;
    return step_dense(layers, L, B, dtype, C, sigma, seed, stream_id0, sq_layers, clip, norms, lanes);
}

int dpclip_step_per_layer(const dpclip_layer* layers, int L, int B, dpclip_dtype dtype, const float* C_layer,
                          float sigma, unsigned long long seed, unsigned long long stream_id0, float* sq_layers,
                          float* clip_layers, float* norms_layers, void* workspace, size_t workspace_bytes,
                          void* stream) {
    if (!layers || L <= 0 || B <= 0 || !C_layer || !sq_layers || !clip_layers) return DPCLIP_ERR_INVALID_ARG;
    if (!(sigma >= 0.f)) return DPCLIP_ERR_INVALID_ARG;
    if (dtype != DPCLIP_F32 && dtype != DPCLIP_BF16) return DPCLIP_ERR_INVALID_ARG;
    double c2 = 0.0;
    for (int l = 0; l < L; ++l) {
        if (!(C_layer[l] > 0.f)) return DPCLIP_ERR_INVALID_ARG;
        c2 += (double)C_layer[l] * C_layer[l];
    }
    const float C_total = (float)sqrt(c2);               // sensitivity of the concatenated clipped gradient
    for (int l = 0; l < L; ++l) {
        const dpclip_layer& y = layers[l];
        if (!y.gW || (y.has_bias && !y.gb)) return DPCLIP_ERR_INVALID_ARG;
        if (y.ldg != y.d_in) return DPCLIP_ERR_UNSUPPORTED;            // noise indexes the dense tensor
    }
    int rc;
    // The stages of the global step with a factor vector per layer: every layer's norms (the layers that go by
    // the Gram identity in one launch), then ALL rows of factors in one launch (row l against C_layer[l]), then
    // the clipped sums -- the wide bf16 layers of one T in one CTA-pair launch, each with its own factor row --
    // with the noise N(0, sigma^2 * sum_l C_l^2).  (Layer after layer, norm -> factors -> clipped sum, so that a
    // layer's second pass finds its inputs in L2, took 566 us on the sequence workload: it gives up both shared
    // launches, and a wide layer's inputs do not fit L2 anyway.)
    constexpr int kMaxTracked = 64;
    int in_gram[kMaxTracked], in_pairs[kMaxTracked];
    const bool track = L <= kMaxTracked;
    if (track) {
        rc = dpclip_gram_layers_sqnorms(layers, L, B, dtype, sq_layers, in_gram, workspace, workspace_bytes, stream);
        if (rc) return rc;
    }
    for (int l = 0; l < L; ++l) {
        const dpclip_layer& y = layers[l];
        if (track && in_gram[l]) continue;
        rc = dpclip_layer_sqnorms(y.A, y.lda, y.Zbar, y.ldz, B, y.T, y.d_in, y.d_out, dtype, y.has_bias,
                                  (dpclip_method)y.method, sq_layers + (size_t)l * B, workspace, workspace_bytes, stream);
        if (rc) return rc;
    }
    if (track) {
        LayerThresholds th;
        for (int l = 0; l < L; ++l) th.C[l] = C_layer[l];
        factors_rows_kernel<<<L, 256, 0, (cudaStream_t)stream>>>(sq_layers, (long)B, B, th, clip_layers, norms_layers);
        if (launch_status()) return DPCLIP_ERR_CUDA;
        rc = shared_clipped_grad_launches(layers, L, B, dtype, clip_layers, (long)B, C_total, sigma, seed, stream_id0,
                                          in_pairs, workspace, workspace_bytes, stream);
        if (rc) return rc;
    } else {
        for (int l = 0; l < L; ++l) {
            rc = dpclip_factors(sq_layers + (size_t)l * B, 1, B, B, C_layer[l], clip_layers + (size_t)l * B,
                                norms_layers ? norms_layers + (size_t)l * B : nullptr, nullptr, stream);
            if (rc) return rc;
        }
    }
    for (int l = 0; l < L; ++l) {
        const dpclip_layer& y = layers[l];
        if (track && in_pairs[l]) continue;
        float* gb = y.has_bias ? y.gb : nullptr;
        NoiseSpec ns = {sigma * C_total, seed, stream_id0 + 2ull * l, stream_id0 + 2ull * l + 1};
        bool noise_done = false;
        rc = clipped_grad_impl(y.A, y.lda, y.Zbar, y.ldz, B, y.T, y.d_in, y.d_out, dtype, clip_layers + (size_t)l * B, y.gW,
                               y.ldg, gb, workspace, workspace_bytes, &ns, &noise_done, (cudaStream_t)stream);
        if (rc) return rc;
        if (!noise_done) {
            rc = dpclip_add_noise(y.gW, (size_t)y.d_out * y.d_in, sigma, C_total, seed, ns.sid_w, stream);
            if (rc) return rc;
            if (gb) {
                rc = dpclip_add_noise(gb, (size_t)y.d_out, sigma, C_total, seed, ns.sid_b, stream);
                if (rc) return rc;
            }
        }
    }
    return DPCLIP_OK;
}

size_t dpclip_model_workspace_bytes(const dpclip_model_layer* layers, int L, int B, dpclip_dtype dtype) {
    size_t ws = kHeaderBytes;
    if (!layers || L <= 0 || L > 256 || B <= 0) return ws;
    {
        dpclip_layer dense[256];
        for (int l = 0; l < L; ++l) {
            if (layers[l].kind == DPCLIP_KIND_DENSE) dense[l] = layers[l].layer;
            else memset(&dense[l], 0, sizeof(dense[l]));
        }
        ws = dpclip_step_workspace_bytes(dense, L, B, dtype);
    }
    for (int l = 0; l < L; ++l) {
        const dpclip_layer& y = layers[l].layer;
        size_t w = kHeaderBytes;
        if (layers[l].kind == DPCLIP_KIND_DENSE)
            w = dpclip_workspace_bytes(B, y.T, y.d_in, y.d_out, dtype, (dpclip_method)y.method);
        else if (layers[l].kind == DPCLIP_KIND_CONV)
            w = dpclip_conv_workspace_bytes(B, &layers[l].conv, y.d_out, dtype, layers[l].z_channel_major);
        if (w > ws) ws = w;
    }
    return ws;
}

int dpclip_model_step(const dpclip_model_layer* layers, int L, int B, dpclip_dtype dtype, float C, float sigma,
                      unsigned long long seed, unsigned long long stream_id0, float* sq_layers, float* clip,
                      float* norms, void* workspace, size_t workspace_bytes, void* stream) {
    int rc = step_args_ok(layers, L, B, dtype, C, sigma, sq_layers, clip);
    if (rc) return rc;
    Lanes lanes;
    one_lane(lanes, workspace, workspace_bytes, stream);
    return step_model(layers, L, B, dtype, C, sigma, seed, stream_id0, sq_layers, clip, norms, lanes);
}

int dpclip_model_step_streams(const dpclip_model_layer* layers, int L, int B, dpclip_dtype dtype, float C, float sigma,
                              unsigned long long seed, unsigned long long stream_id0, float* sq_layers, float* clip,
                              float* norms, int n_streams, void* const* streams, void* const* workspaces,
                              size_t workspace_bytes) {
    int rc = step_args_ok(layers, L, B, dtype, C, sigma, sq_layers, clip);
    if (rc) return rc;
    Lanes lanes;
    if ((rc = many_lanes(lanes, n_streams, streams, workspaces, workspace_bytes))) return rc;
    return step_model(layers, L, B, dtype, C, sigma, seed, stream_id0, sq_layers, clip, norms, lanes);
}

size_t dpclip_step_host_arena_bytes(const dpclip_layer* layers, int L, int B, dpclip_dtype dtype) {
    if (!layers || L <= 0 || B <= 0) return 0;
    const size_t es = elt_size(dtype);
    size_t ws = dpclip_step_workspace_bytes(layers, L, B, dtype), total = 0;
    for (int l = 0; l < L; ++l) {
        const dpclip_layer& y = layers[l];
        total += round_up((size_t)B * y.T * y.d_in * es, 256);
        total += round_up((size_t)B * y.T * y.d_out * es, 256);
        total += round_up((size_t)y.d_out * y.d_in * 4, 256);
        total += round_up((size_t)y.d_out * 4, 256);
    }
    total += round_up(ws, 256);
    total += round_up((size_t)L * B * 4, 256) + 2 * round_up((size_t)B * 4, 256);
    return total;
}

int dpclip_step_host(const dpclip_layer* layers, int L, int B, dpclip_dtype dtype, float C, float sigma,
                     unsigned long long seed, unsigned long long stream_id0, float* host_clip,
                     float* host_norms, void* arena, size_t arena_bytes, void* stream) {
    if (!layers || L <= 0 || L > 64 || B <= 0 || !arena) return DPCLIP_ERR_INVALID_ARG;
    if (!aligned_to(arena, 256)) return DPCLIP_ERR_MISALIGNED;
    if (arena_bytes < dpclip_step_host_arena_bytes(layers, L, B, dtype)) return DPCLIP_ERR_WORKSPACE;
    cudaStream_t st = (cudaStream_t)stream;
    const size_t es = elt_size(dtype);
    char* cur = static_cast<char*>(arena);
    auto take = [&](size_t bytes) { char* p = cur; cur += round_up(bytes, 256); return (void*)p; };

    const size_t ws_bytes = dpclip_step_workspace_bytes(layers, L, B, dtype);
    for (int l = 0; l < L; ++l) {
        const dpclip_layer& y = layers[l];
        if (y.lda != y.d_in || y.ldz != y.d_out || y.ldg != y.d_in) return DPCLIP_ERR_INVALID_ARG;
        if (!y.A || !y.Zbar || !y.gW || (y.has_bias && !y.gb)) return DPCLIP_ERR_INVALID_ARG;
    }
    void* ws = take(ws_bytes);
    float* sq = (float*)take((size_t)L * B * 4);
    if (dpclip_workspace_init(ws, ws_bytes, stream)) return DPCLIP_ERR_CUDA;

    // Arena: [workspace][sq][A_0][Zb_0][A_1][Zb_1]...[gW_0][gb_0][gW_1]...[clip][norms], every tensor on
    // the next 256-byte boundary.  When the host tensors of a direction sit back to back in the same
    // order with the same padding (one pinned buffer carved up this way), that direction is ONE copy.
    dpclip_layer dev[64];
    char* in_begin = cur;
    bool in_packed = true;
    const char* h_in0 = static_cast<const char*>(layers[0].A);
    for (int l = 0; l < L; ++l) {
        const dpclip_layer& y = layers[l];
        dev[l] = y;
        const size_t a_bytes = (size_t)B * y.T * y.d_in * es, z_bytes = (size_t)B * y.T * y.d_out * es;
        dev[l].A = take(a_bytes);
        dev[l].Zbar = take(z_bytes);
        in_packed = in_packed && static_cast<const char*>(y.A) - h_in0 == static_cast<const char*>(dev[l].A) - in_begin &&
                    static_cast<const char*>(y.Zbar) - h_in0 == static_cast<const char*>(dev[l].Zbar) - in_begin;
    }
    // a merged copy ends where the last tensor really ends: the host buffer need not extend to the padded end
    const size_t in_bytes = (size_t)(static_cast<const char*>(dev[L - 1].Zbar) - in_begin) +
                            (size_t)B * layers[L - 1].T * layers[L - 1].d_out * es;
    char* out_begin = cur;
    bool out_packed = true;
    const char* h_out0 = reinterpret_cast<const char*>(layers[0].gW);
    for (int l = 0; l < L; ++l) {
        const dpclip_layer& y = layers[l];
        dev[l].gW = (float*)take((size_t)y.d_out * y.d_in * 4);
        dev[l].gb = (float*)take((size_t)y.d_out * 4);
        out_packed = out_packed && reinterpret_cast<const char*>(y.gW) - h_out0 == reinterpret_cast<const char*>(dev[l].gW) - out_begin &&
                     (!y.has_bias || reinterpret_cast<const char*>(y.gb) - h_out0 == reinterpret_cast<const char*>(dev[l].gb) - out_begin);
        if (!y.has_bias) dev[l].gb = nullptr;
    }
    float* clip = (float*)take((size_t)B * 4);
    float* norms = (float*)take((size_t)B * 4);
    out_packed = out_packed && host_clip && host_norms &&
                 reinterpret_cast<const char*>(host_clip) - h_out0 == reinterpret_cast<const char*>(clip) - out_begin &&
                 reinterpret_cast<const char*>(host_norms) - h_out0 == reinterpret_cast<const char*>(norms) - out_begin;
    const size_t out_bytes = (size_t)(reinterpret_cast<const char*>(norms) - out_begin) + (size_t)B * 4;

    if (in_packed) {
        if (cudaMemcpyAsync(in_begin, h_in0, in_bytes, cudaMemcpyHostToDevice, st) != cudaSuccess) return DPCLIP_ERR_CUDA;
    } else {
        for (int l = 0; l < L; ++l) {
            const dpclip_layer& y = layers[l];
            const size_t a_bytes = (size_t)B * y.T * y.d_in * es, z_bytes = (size_t)B * y.T * y.d_out * es;
            if (cudaMemcpyAsync(const_cast<void*>(dev[l].A), y.A, a_bytes, cudaMemcpyHostToDevice, st) != cudaSuccess ||
                cudaMemcpyAsync(const_cast<void*>(dev[l].Zbar), y.Zbar, z_bytes, cudaMemcpyHostToDevice, st) != cudaSuccess)
                return DPCLIP_ERR_CUDA;
        }
    }
    int rc = dpclip_step(dev, L, B, dtype, C, sigma, seed, stream_id0, sq, clip, norms, ws, ws_bytes, stream);
    if (rc) return rc;
    if (out_packed) {
        if (cudaMemcpyAsync(const_cast<char*>(h_out0), out_begin, out_bytes, cudaMemcpyDeviceToHost, st) != cudaSuccess)
            return DPCLIP_ERR_CUDA;
        return DPCLIP_OK;
    }
    for (int l = 0; l < L; ++l) {
        const dpclip_layer& y = layers[l];
        if (cudaMemcpyAsync(y.gW, dev[l].gW, (size_t)y.d_out * y.d_in * 4, cudaMemcpyDeviceToHost, st) !=
            cudaSuccess) return DPCLIP_ERR_CUDA;
        if (y.has_bias &&
            cudaMemcpyAsync(y.gb, dev[l].gb, (size_t)y.d_out * 4, cudaMemcpyDeviceToHost, st) != cudaSuccess)
            return DPCLIP_ERR_CUDA;
    }
    if (host_clip && cudaMemcpyAsync(host_clip, clip, (size_t)B * 4, cudaMemcpyDeviceToHost, st) != cudaSuccess)
        return DPCLIP_ERR_CUDA;
    if (host_norms && cudaMemcpyAsync(host_norms, norms, (size_t)B * 4, cudaMemcpyDeviceToHost, st) != cudaSuccess)
        return DPCLIP_ERR_CUDA;
    return DPCLIP_OK;
}


// ---------------------------------------------------------------------------
// Clipped sum without a caller-provided workspace.
//
// Some callers have no way to hand this library device memory: a plug-in that runs inside a host
// application which owns every byte of the GPU, a service whose memory pool is carved up once at
// start-up, or code that is already inside a region where cudaMalloc is not permitted.  For them
// the split-row scratch of dpclip_clipped_grad lives in the fixed array below instead.  The array
// is part of the loaded library image: every GPU that loads libdpclip holds these 16 MB (+ 256 bytes)
// until the process exits, whether or not this entry point is ever called.
// ---------------------------------------------------------------------------
constexpr size_t kStaticScratchBytes = (size_t)16 << 20;
static __device__ __align__(256) unsigned char g_static_scratch[kHeaderBytes + kStaticScratchBytes];

// In host code `g_static_scratch` is only a handle for the runtime, not a device address, so the
// address is looked up once per device (with that device current) and remembered.
static void* static_scratch_for_current_device(int* rc) {
    // two host threads may make the first call on a device at once: both look the same address up,
    // and the slot is published with an atomic store
    static std::atomic<void*> cached[64];
    int dev = -1;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= 64) { *rc = DPCLIP_ERR_CUDA; return nullptr; }
    void* ptr = cached[dev].load(std::memory_order_acquire);
    if (!ptr) {
        if (cudaGetSymbolAddress(&ptr, g_static_scratch) != cudaSuccess || !ptr) { *rc = DPCLIP_ERR_CUDA; return nullptr; }
        cached[dev].store(ptr, std::memory_order_release);
    }
    *rc = DPCLIP_OK;
    return ptr;
}

size_t dpclip_noalloc_max_output_bytes(void) { return kStaticScratchBytes / 2; }

int dpclip_clipped_grad_noalloc(const void* A, long lda, const void* Zbar, long ldz, int B, int T, int d_in,
                                int d_out, dpclip_dtype dtype, const float* clip, float* gW, long ldg, float* gb,
                                void* stream) {
    int rc = check_layer_args(A, lda, Zbar, ldz, B, T, d_in, d_out, dtype);
    if (rc) return rc;
    if (!gW || ldg < d_in) return DPCLIP_ERR_INVALID_ARG;
    if (!aligned_to(gW, 4) || (gb && !aligned_to(gb, 4))) return DPCLIP_ERR_MISALIGNED;
    // The output, padded to 256 x 256 tiles, may take at most half of the array: room for one partial tile per
    // output tile and about as many again for the row split, which is clamped to what the array holds (at the
    // limit: 16 tiles of 512 x 256, 31 partial tiles, so 15 pairs of SMs instead of 74 -- correct, slower).
    const size_t padded = (size_t)ceil_div(d_out, 256) * 256 * ((size_t)ceil_div(d_in, 256) * 256) * 4;
    if (padded > dpclip_noalloc_max_output_bytes()) return DPCLIP_ERR_WORKSPACE;
    void* scratch = static_scratch_for_current_device(&rc);
    if (rc) return rc;
    cudaStream_t st = (cudaStream_t)stream;
    // the array keeps whatever the previous call left: the status header has to start at zero (the
    // partial tiles need no clearing, every tile that is read is written first)
    if (cudaMemsetAsync(scratch, 0, kHeaderBytes, st) != cudaSuccess) return DPCLIP_ERR_CUDA;
    if (tc_eligible(A, lda, Zbar, ldz, dtype))
        return launch_zta_tc(A, lda, Zbar, ldz, B, T, d_in, d_out, false, 0, clip, gW, ldg, gb, nullptr, scratch,
                             kHeaderBytes + kStaticScratchBytes, nullptr, nullptr, st, /*fit_to_workspace=*/true);
    return launch_simt_grad(A, lda, Zbar, ldz, B, T, d_in, d_out, dtype, clip, gW, ldg, gb, st);
}

}  // extern "C"
