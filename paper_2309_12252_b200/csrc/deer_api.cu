// C-ABI entry points of the DEER-GRU library: validation, workspace carving,
// kernel sequencing and the Newton loop control.
#include <math.h>
#include <stdio.h>
#include <string.h>
#include <stdlib.h>

#include <algorithm>
#include <map>
#include <mutex>
#include <string>
#include <vector>

#include "common.cuh"
#include "kernels_generic.cuh"
#include "scan_onepass.cuh"
#include "scan_hold4.cuh"
#include "scan_warp8.cuh"
#include "scan_warpn.cuh"
#include "scan_warpn_fused.cuh"
#include "scan_fused_fwd.cuh"
#include "scan_cta64.cuh"
#include "scan_umma64.cuh"
#include "scan_fused_fwd64.cuh"
#include "cell_wide.cuh"
#include "vjp_wide.cuh"

namespace deer {

std::atomic<long long> g_launches{0};
static thread_local char t_err[256] = "";

void set_error(cudaError_t e, const char *where)
{
    snprintf(t_err, sizeof(t_err), "%s: %s", where, cudaGetErrorString(e));
}

// ---- per-kernel profiling (off by default; benchmarks switch it on for a separate pass)
struct ProfRec { const char *name; cudaEvent_t e0, e1; };
static std::mutex g_prof_mu;
static std::atomic<bool> g_prof_on{false};
static std::vector<ProfRec> g_prof;

KernelScope::KernelScope(const char *name_, cudaStream_t st_) : name(name_), st(st_)
{
    if (!g_prof_on.load(std::memory_order_relaxed)) return;
    if (cudaEventCreate(&e0) != cudaSuccess || cudaEventCreate(&e1) != cudaSuccess) { e0 = e1 = nullptr; return; }
    cudaEventRecord(e0, st);
}

KernelScope::~KernelScope()
{
    if (!e0) return;
    cudaEventRecord(e1, st);
    std::lock_guard<std::mutex> lk(g_prof_mu);
    g_prof.push_back({name, e0, e1});
}

// Bump allocator over the caller's workspace; with base == nullptr it only measures.
struct Carver {
    char *base;
    size_t off = 0;
    explicit Carver(void *b) : base((char *)b) {}
    template <typename T> T *take(size_t count)
    {
        size_t o = off;
        off = align_up(off + count * sizeof(T));
        return base ? (T *)(base + o) : nullptr;
    }
};

static int gen_chunk_len(int T)
{
    int L = (int)ceil(sqrt((double)T));
    if (L < 16) L = 16;
    if (L > 256) L = 256;
    return L;
}

struct ScanWs {
    float *carA, *carB, *starts;
    int L, nch;
    OnePassWs op;        // single-pass path (n in {1,2,4,8}); op.nch == 0 when not applicable
};

static int num_sms();

static bool onepass_ll_aggs(int n) { return n <= 4; }

static int onepass_tile_len(int n, int B, int T, int *sw)
{
    *sw = 0;
    switch (n) {
    case 1: return OnePass<1>::L;
    case 2: return OnePass<2>::L;
    case 4: return OnePass<4>::L;
    case 8: *sw = Warp8::chain_len(B, T, 4 * num_sms()); return Warp8::WARPS * *sw;
    case 16: *sw = WarpN<16>::chain_len(B, T, WarpN<16>::CTAS_PER_SM * num_sms()); return WarpN<16>::WARPS * *sw;
    case 32: *sw = WarpN<32>::chain_len(B, T, WarpN<32>::CTAS_PER_SM * num_sms()); return WarpN<32>::WARPS * *sw;
    case 64: return Cta64::L;
    default: return 0;
    }
}

static ScanWs carve_scan(Carver &cv, int B, int T, int n)
{
    ScanWs w;
    w.L = gen_chunk_len(T);
    w.nch = (T + w.L - 1) / w.L;
    w.carA = cv.take<float>((size_t)B * w.nch * n * n);
    w.carB = cv.take<float>((size_t)B * w.nch * n);
    w.starts = cv.take<float>((size_t)B * w.nch * n);
    w.op = OnePassWs{};
    int L1 = onepass_tile_len(n, B, T, &w.op.sw);
    if (L1) {
        w.op.nch = (T + L1 - 1) / L1;
        size_t tiles = (size_t)B * w.op.nch;
        w.op.flags = cv.take<unsigned>(tiles);
        // (n <= 4 publish their aggregates as 64-bit {value, flag} words)
        w.op.aggs = cv.take<float>(tiles * (n * n + n) * (onepass_ll_aggs(n) ? 2 : 1));
        w.op.starts = cv.take<unsigned long long>(tiles * n);
        w.op.pfx = nullptr;
        if (n == 16) w.op.pfx = cv.take<float>(tiles * (FusedFwd<16>::WARPS - 1) * FusedFwd<16>::AGG);
        if (n == 32) w.op.pfx = cv.take<float>(tiles * (FusedFwd<32>::WARPS - 1) * FusedFwd<32>::AGG);
    }
    return w;
}

constexpr int MAX_DEVICES = 64;
static int g_num_sms[MAX_DEVICES] = {0};
static int num_sms()
{
    int dev = 0;
    cudaGetDevice(&dev);
    if (dev < 0 || dev >= MAX_DEVICES) dev = 0;
    if (!g_num_sms[dev]) {
        int v = 0;
        cudaDeviceGetAttribute(&v, cudaDevAttrMultiProcessorCount, dev);
        g_num_sms[dev] = v > 0 ? v : 148;
    }
    return g_num_sms[dev];
}

// Clears the single-pass scan's flag / state words and counters (needed once per workspace: the
// scans leave them cleared).
static int scan_prep(const ScanArgs &a, const OnePassWs &w, cudaStream_t st)
{
    const size_t tiles = (size_t)a.B * w.nch;
    const size_t agg_words = onepass_ll_aggs(a.n) ? tiles * (size_t)(a.n * a.n + a.n) : 0;
    const size_t words = tiles * (size_t)(a.n + 1) + agg_words;
    unsigned pb = (unsigned)((words + 255) / 256);
    if (pb > 592u) pb = 592u;
    if (pb < 1u) pb = 1u;
    DEER_KERNEL("scan_prep_kernel", st, scan_prep_kernel<<<pb, 256, 0, st>>>(a.st, w.flags, tiles, w.starts, tiles * (size_t)a.n,
                                                      (unsigned long long *)w.aggs, agg_words));
    return DEER_OK;
}

// Resolver warps per resolver CTA x sequences one warp can serve, for the kernel that scans size n.
static int resolver_cta_capacity(int n, bool umma)
{
    switch (n) {
    case 1: return OnePass<1>::WARPS * OnePass<1>::MAX_SEQ_PER_WARP;
    case 2: return OnePass<2>::WARPS * OnePass<2>::MAX_SEQ_PER_WARP;
    case 4: return OnePass<4>::WARPS * OnePass<4>::MAX_SEQ_PER_WARP;
    case 8: return Warp8::RES_WARPS * OnePass<8>::MAX_SEQ_PER_WARP;
    case 16: return WarpN<16>::RES_WARPS * WarpN<16>::MAX_SEQ_PER_WARP;
    case 32: return WarpN<32>::RES_WARPS * WarpN<32>::MAX_SEQ_PER_WARP;
    case 64: return umma ? Umma64::RES_WARPS * Umma64::MAX_SEQ_PER_WARP : Cta64::RES_WARPS * Cta64::MAX_SEQ_PER_WARP;
    default: return 0;
    }
}

// Resolver CTAs of a single-pass launch: one warp per sequence up to res_cap CTAs, then several
// sequences per warp, and as many CTAs as the batch needs at max_seq_per_warp sequences per warp.
static int resolver_ctas(int B, int res_warps, int max_seq_per_warp, int res_cap)
{
    int R = (B + res_warps - 1) / res_warps;
    if (R > res_cap) R = res_cap;
    const int per_cta_cap = res_warps * max_seq_per_warp;
    const int need = (B + per_cta_cap - 1) / per_cta_cap;
    return need > R ? need : R;
}

// Resolver CTAs only spin; the workers that feed them must be resident beside them.  At least one CTA
// per SM is resident whatever the kernel, so the single-pass path is taken only while the resolvers a
// batch needs fit a quarter of the SMs; larger batches use the three-level scan.
static long long single_pass_max_batch(int n, bool umma)
{
    return (long long)(num_sms() / 4) * resolver_cta_capacity(n, umma);
}

// n = 16, 32: warps of a resolver CTA that resolve.  A resolver CTA's staging area is shared by its resolving warps,
// and the walk over ONE sequence's tiles is the serial part of a scan: small batches give each sequence a deeper ring.
static int big_res_warps(int B) { return B <= 4 ? 1 : B <= 8 ? 2 : 4; }
// n = 64 (two resolving warps per CTA at most): one warp with all the CTA's tile slots for small batches
static int res_warps64(int B) { return B <= 8 ? 1 : 2; }

struct PassCfg {
    const char *name;
    int threads;
    size_t smem;
    int res_warps;          // resolver warps per resolver CTA
    int max_seq_per_warp;
    int cta_cap;            // CTAs per SM at most
    int res_cap;            // resolver CTAs before warps take several sequences
};

// One persistent launch: grid = resident CTAs (or fewer when there are few tiles); the first
// `resolvers` role tickets become resolver CTAs.
template <typename Kern>
static int launch_single_pass(Kern kern, int (&occ_dev)[MAX_DEVICES], const PassCfg &c, ScanArgs a, OnePassWs w, bool prep,
                              cudaStream_t st)
{
    // the shared-memory opt-in and the occupancy are per device: looked up on each device's first launch
    int dev = 0;
    cudaGetDevice(&dev);
    if (dev < 0 || dev >= MAX_DEVICES) dev = 0;
    int &occ = occ_dev[dev];
    if (!occ) {
        cudaError_t e = cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)c.smem);
        if (e != cudaSuccess) { set_error(e, "cudaFuncSetAttribute(single-pass scan)"); return DEER_ERR_CUDA; }
        int o = 0;
        e = cudaOccupancyMaxActiveBlocksPerMultiprocessor(&o, kern, c.threads, c.smem);
        if (e != cudaSuccess || o < 1) { set_error(e, "occupancy(single-pass scan)"); return DEER_ERR_CUDA; }
        occ = o < c.cta_cap ? o : c.cta_cap;
    }
    const size_t tiles = (size_t)a.B * w.nch;
    const size_t resident = (size_t)num_sms() * occ;
    const int R = resolver_ctas(a.B, c.res_warps, c.max_seq_per_warp, c.res_cap);
    if ((size_t)R * 4 > resident) {      // (scan_is_single_pass keeps such batches off this path)
        snprintf(t_err, sizeof(t_err), "single-pass scan: %d resolver CTAs for %zu resident", R, resident);
        return DEER_ERR_INVALID_ARG;
    }
    w.resolvers = R;
    const size_t want = tiles + (size_t)R;
    unsigned grid = (unsigned)(want < resident ? want : resident);
    if (grid < (unsigned)R + 1u) grid = (unsigned)R + 1u;
    int Wd = 8;
    if (Wd > w.nch) Wd = w.nch;
    w.Wd = Wd;
    w.nwin = (w.nch + Wd - 1) / Wd;
    w.total_ids = (unsigned)((size_t)w.nwin * a.B * Wd);
    int rc;
    if (prep && (rc = scan_prep(a, w, st)) != DEER_OK) return rc;
    DEER_KERNEL_PDL(c.name, a.n <= 8, st, kern, grid, (unsigned)c.threads, c.smem, a, w);
    return DEER_OK;
}

template <int N, bool REV>
static int launch_onepass(ScanArgs a, OnePassWs w, bool prep, cudaStream_t st)
{
    using C = OnePass<N>;
    static int occ[MAX_DEVICES] = {0};
    const PassCfg c{"scan_onepass_kernel", C::THREADS, C::SMEM, C::WARPS, C::MAX_SEQ_PER_WARP, 32, 8};
    return launch_single_pass(scan_onepass_kernel<N, REV>, occ, c, a, w, prep, st);
}

template <bool REV>
static int launch_hold4(ScanArgs a, OnePassWs w, bool prep, cudaStream_t st)
{
    using C = OnePass<4>;
    static int occ[MAX_DEVICES] = {0};
    const PassCfg c{"scan_hold4_kernel", C::THREADS, Hold4::SMEM, C::WARPS, C::MAX_SEQ_PER_WARP, 32, 8};
    return launch_single_pass(scan_hold4_kernel<REV>, occ, c, a, w, prep, st);
}

template <bool REV>
static int launch_warp8(ScanArgs a, OnePassWs w, bool prep, cudaStream_t st)
{
    using C = Warp8;
    static int occ[MAX_DEVICES] = {0};
    const PassCfg c{"scan_warp8_kernel", C::THREADS, C::SMEM, C::RES_WARPS, OnePass<8>::MAX_SEQ_PER_WARP, 4, 8};
    return launch_single_pass(scan_warp8_kernel<REV>, occ, c, a, w, prep, st);
}

template <int N, bool REV>
static int launch_warpn(ScanArgs a, OnePassWs w, bool prep, cudaStream_t st)
{
    using C = WarpN<N>;
    static int occ[MAX_DEVICES] = {0};
    w.res_warps = big_res_warps(a.B);
    const PassCfg c{"scan_warpn_kernel", C::THREADS, C::SMEM, w.res_warps, C::MAX_SEQ_PER_WARP, 8, 8};
    return launch_single_pass(scan_warpn_kernel<N, REV>, occ, c, a, w, prep, st);
}

// scans that generate J_t from coefficient rows (a.J) and a.Wh
template <int N, bool REV>
static int launch_warpnf(ScanArgs a, OnePassWs w, bool prep, cudaStream_t st)
{
    using C = WarpNF<N, REV>;
    static int occ[MAX_DEVICES] = {0};
    w.res_warps = big_res_warps(a.B);
    const PassCfg c{"scan_warpnf_kernel", C::THREADS, C::SMEM, w.res_warps, C::MAX_SEQ_PER_WARP, 8, 8};
    return launch_single_pass(scan_warpnf_kernel<N, REV>, occ, c, a, w, prep, st);
}

// forward scan of deer_gru_eval in the Newton-update form, two launches: chunk reduce + carries, then the
// replay of all chains (16 per warp in lockstep)
template <int N>
static int launch_fused_fwd(ScanArgs a, OnePassWs w, bool prep, cudaStream_t st)
{
    using C = FusedFwd<N>;
    static int occ[MAX_DEVICES] = {0};
    static int occ_apply[MAX_DEVICES] = {0};
    w.res_warps = big_res_warps(a.B);
    const PassCfg c{"scan_fused_reduce_kernel", C::THREADS, C::SMEM, w.res_warps, C::MAX_SEQ_PER_WARP, 8, 8};
    int rc = launch_single_pass(scan_fused_reduce_kernel<N>, occ, c, a, w, prep, st);
    if (rc != DEER_OK) return rc;
    int dev = 0;
    cudaGetDevice(&dev);
    if (dev < 0 || dev >= MAX_DEVICES) dev = 0;
    if (!occ_apply[dev]) {
        cudaError_t e = cudaFuncSetAttribute(scan_fused_apply_kernel<N>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)C::A_SMEM);
        if (e != cudaSuccess) { set_error(e, "cudaFuncSetAttribute(scan apply)"); return DEER_ERR_CUDA; }
        int o = 0;
        e = cudaOccupancyMaxActiveBlocksPerMultiprocessor(&o, scan_fused_apply_kernel<N>, C::A_THREADS, C::A_SMEM);
        if (e != cudaSuccess || o < 1) { set_error(e, "occupancy(scan apply)"); return DEER_ERR_CUDA; }
        occ_apply[dev] = o;
    }
    const long long nchain = (a.T + w.sw - 1) / w.sw;
    const long long groups = ((long long)a.B * nchain + C::ROWS - 1) / C::ROWS;
    const long long want = (groups + C::A_WARPS - 1) / C::A_WARPS;
    const long long resident = (long long)num_sms() * occ_apply[dev];
    const unsigned grid = (unsigned)(want < resident ? want : resident);
    DEER_KERNEL_PDL("scan_fused_apply_kernel", false, st, scan_fused_apply_kernel<N>, grid, (unsigned)C::A_THREADS, C::A_SMEM, a, w);
    return DEER_OK;
}

// n = 64: the same two launches (a CTA of four warps per chain; the replay kernel reads W_h^T from shared memory)
static int launch_fused_fwd64(ScanArgs a, OnePassWs w, bool prep, cudaStream_t st)
{
    using C = FusedFwd<64>;
    static int occ[MAX_DEVICES] = {0};
    static int occ_apply[MAX_DEVICES] = {0};
    w.sw = C::L;                               // a tile is one chain
    w.res_warps = res_warps64(a.B);
    const PassCfg c{"scan_fused_reduce64_kernel", C::THREADS, C::SMEM, w.res_warps, C::MAX_SEQ_PER_WARP, 4, 16};
    int rc = launch_single_pass(scan_fused_reduce64_kernel, occ, c, a, w, prep, st);
    if (rc != DEER_OK) return rc;
    int dev = 0;
    cudaGetDevice(&dev);
    if (dev < 0 || dev >= MAX_DEVICES) dev = 0;
    if (!occ_apply[dev]) {
        cudaError_t e = cudaFuncSetAttribute(scan_fused_apply64_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)C::P_SMEM);
        if (e != cudaSuccess) { set_error(e, "cudaFuncSetAttribute(scan apply)"); return DEER_ERR_CUDA; }
        int o = 0;
        e = cudaOccupancyMaxActiveBlocksPerMultiprocessor(&o, scan_fused_apply64_kernel, C::P_THREADS, C::P_SMEM);
        if (e != cudaSuccess || o < 1) { set_error(e, "occupancy(scan apply)"); return DEER_ERR_CUDA; }
        occ_apply[dev] = o;
    }
    const long long nchain = (a.T + w.sw - 1) / w.sw;
    const long long groups = ((long long)a.B * nchain + C::ROWS - 1) / C::ROWS;
    const long long want = (groups + C::P_PAIRS - 1) / C::P_PAIRS;
    const long long resident = (long long)num_sms() * occ_apply[dev];
    const unsigned grid = (unsigned)(want < resident ? want : resident);
    DEER_KERNEL_PDL("scan_fused_apply_kernel", false, st, scan_fused_apply64_kernel, grid, (unsigned)C::P_THREADS, C::P_SMEM, a, w);
    return DEER_OK;
}

template <bool REV>
static int launch_cta64(ScanArgs a, OnePassWs w, bool prep, cudaStream_t st)
{
    using C = Cta64;
    static int occ[MAX_DEVICES] = {0};
    w.res_warps = res_warps64(a.B);
    const PassCfg c{"scan_cta64_kernel", C::THREADS, C::SMEM, w.res_warps, C::MAX_SEQ_PER_WARP, 8, 16};
    return launch_single_pass(scan_cta64_kernel<REV>, occ, c, a, w, prep, st);
}

template <bool REV>
static int launch_umma64(ScanArgs a, OnePassWs w, bool prep, cudaStream_t st)
{
    using C = Umma64;
    static int occ[MAX_DEVICES] = {0};
    w.res_warps = C::RES_WARPS;
    const PassCfg c{"scan_umma64_kernel", C::THREADS, C::SMEM, C::RES_WARPS, C::MAX_SEQ_PER_WARP, 2, 8};
    return launch_single_pass(scan_umma64_kernel<REV>, occ, c, a, w, prep, st);
}

static int scan_onepass(ScanArgs a, OnePassWs w, bool prep, int flags, cudaStream_t st)
{
    const bool umma = (flags & DEER_FLAG_TCGEN05) != 0;
    switch (a.n * 2 + (a.reverse ? 1 : 0)) {
    case 2: return launch_onepass<1, false>(a, w, prep, st);
    case 3: return launch_onepass<1, true>(a, w, prep, st);
    case 4: return launch_onepass<2, false>(a, w, prep, st);
    case 5: return launch_onepass<2, true>(a, w, prep, st);
    case 8: return launch_hold4<false>(a, w, prep, st);
    case 9: return launch_hold4<true>(a, w, prep, st);
    case 16: return launch_warp8<false>(a, w, prep, st);
    case 17: return launch_warp8<true>(a, w, prep, st);
    case 32: return a.Wh ? (a.residual ? launch_fused_fwd<16>(a, w, prep, st) : launch_warpnf<16, false>(a, w, prep, st))
                         : launch_warpn<16, false>(a, w, prep, st);
    case 33: return a.Wh ? launch_warpnf<16, true>(a, w, prep, st) : launch_warpn<16, true>(a, w, prep, st);
    case 64: return a.Wh ? (a.residual ? launch_fused_fwd<32>(a, w, prep, st) : launch_warpnf<32, false>(a, w, prep, st))
                         : launch_warpn<32, false>(a, w, prep, st);
    case 65: return a.Wh ? launch_warpnf<32, true>(a, w, prep, st) : launch_warpn<32, true>(a, w, prep, st);
    case 128: return umma ? launch_umma64<false>(a, w, prep, st)
                          : (a.Wh && a.residual) ? launch_fused_fwd64(a, w, prep, st) : launch_cta64<false>(a, w, prep, st);
    case 129: return umma ? launch_umma64<true>(a, w, prep, st) : launch_cta64<true>(a, w, prep, st);
    default: return DEER_ERR_UNSUPPORTED_N;
    }
}

static int opt_in_smem(const void *fn, size_t bytes)
{
    if (bytes > 48 * 1024) {
        cudaError_t e = cudaFuncSetAttribute(fn, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)bytes);
        if (e != cudaSuccess) { set_error(e, "cudaFuncSetAttribute"); return DEER_ERR_CUDA; }
    }
    return DEER_OK;
}

// Three-level scan with the generic kernels.
static int scan_generic(ScanArgs a, cudaStream_t st)
{
    const int n = a.n, nn = n * n;
    size_t sm_red = sizeof(float) * (3 * nn + 2 * n);
    size_t sm_car = sizeof(float) * (nn + n);
    int rc;
    if ((rc = opt_in_smem((const void *)gen_reduce_kernel, sm_red)) != DEER_OK) return rc;
    dim3 grid(a.nch, a.B);
    if (a.nch > 1) {
        DEER_KERNEL("gen_reduce_kernel", st, gen_reduce_kernel<<<grid, GEN_THREADS, sm_red, st>>>(a));
    }
    DEER_KERNEL("gen_carry_kernel", st, gen_carry_kernel<<<a.B, GEN_THREADS, sm_car, st>>>(a));
    DEER_KERNEL("gen_apply_kernel", st, gen_apply_kernel<<<grid, GEN_THREADS, sm_car, st>>>(a));
    return DEER_OK;
}

static bool scan_is_single_pass(const ScanArgs &a, const ScanWs &w, int flags)
{
    const bool aligned = (((uintptr_t)a.J | (uintptr_t)a.b | (uintptr_t)a.y) & 15) == 0;
    return !(flags & DEER_FLAG_GENERIC) && w.op.nch > 0 && aligned &&
           a.B <= single_pass_max_batch(a.n, (flags & DEER_FLAG_TCGEN05) != 0);
}

// prep: clear the single-pass scan's words first (false when the previous scan on this workspace
// left them cleared)
static void apply_test_flags(ScanArgs &a, int flags)
{
    if (flags & DEER_FLAG_EXPIRE_WAITS) { a.spin_limit = 4u; a.no_resolve = 1; }
}

static int run_scan(ScanArgs a, const ScanWs &w, int flags, cudaStream_t st, bool prep = true)
{
    apply_test_flags(a, flags);
    if (scan_is_single_pass(a, w, flags)) return scan_onepass(a, w.op, prep, flags, st);
    return scan_generic(a, st);
}

// tensor-core affine map (K = inputs, nout = outputs; see affine_mma_kernel)
template <int NB_MAX, bool WT>
static int launch_affine_mma(const float *in, const float *W, const float *bias, float *out, size_t N, int K, int nout,
                             cudaStream_t st)
{
    const size_t sm = sizeof(float) * 2 * (size_t)K * (nout + 4);
    int rc;
    if ((rc = opt_in_smem((const void *)affine_mma_kernel<NB_MAX, WT>, sm)) != DEER_OK) return rc;
    const size_t tiles = (N + 127) / 128;
    const size_t per_sm = sm > 110 * 1024 ? 1 : 2;
    const size_t cap = (size_t)num_sms() * per_sm;
    const unsigned blocks = (unsigned)(tiles < cap ? tiles : cap);
    DEER_KERNEL("affine_mma_kernel", st, (affine_mma_kernel<NB_MAX, WT><<<blocks, 256, sm, st>>>(in, W, bias, out, N, K, nout)));
    return DEER_OK;
}

// out[e][g] = bias[g] + sum_k W[g][k] in[e][k]   (wt_given: W is stored [k][g]; bias may be null)
static int run_affine(const float *in, const float *W, const float *bias, float *out, size_t N, int m, int n3,
                      int wt_given, cudaStream_t st)
{
    // tensor-core path: K and the output count multiples of 8, 8-byte aligned rows, weights fit shared memory
    const bool aligned8 = (((uintptr_t)in | (uintptr_t)out) & 7) == 0;
    if (aligned8 && m % 8 == 0 && m >= 16 && n3 % 8 == 0 && n3 <= 192 &&
        sizeof(float) * 2 * (size_t)m * (n3 + 4) <= 200 * 1024) {
        if (n3 <= 64) return wt_given ? launch_affine_mma<8, true>(in, W, bias, out, N, m, n3, st)
                                      : launch_affine_mma<8, false>(in, W, bias, out, N, m, n3, st);
        if (n3 <= 96) return wt_given ? launch_affine_mma<12, true>(in, W, bias, out, N, m, n3, st)
                                      : launch_affine_mma<12, false>(in, W, bias, out, N, m, n3, st);
        return wt_given ? launch_affine_mma<24, true>(in, W, bias, out, N, m, n3, st)
                        : launch_affine_mma<24, false>(in, W, bias, out, N, m, n3, st);
    }
    int G = 256 / n3;
    while (G > 1 && sizeof(float) * (size_t)G * PROJ_PP * (m + 1) > 64 * 1024) --G;
    const size_t sm = sizeof(float) * ((size_t)m * n3 + (size_t)G * PROJ_PP * (m + 1));
    if (G < 1 || sm > 200 * 1024) return DEER_ERR_UNSUPPORTED_N;
    int rc;
    if ((rc = opt_in_smem((const void *)proj_tiled_kernel, sm)) != DEER_OK) return rc;
    const size_t tiles = (N + (size_t)G * PROJ_PP - 1) / ((size_t)G * PROJ_PP);
    const size_t cap = (size_t)num_sms() * 8;
    const unsigned blocks = (unsigned)(tiles < cap ? tiles : cap);
    const int threads = (n3 * G + 31) / 32 * 32;
    DEER_KERNEL("proj_tiled_kernel", st,
                proj_tiled_kernel<<<blocks, threads, sm, st>>>(in, W, bias, out, N, m, n3, G, wt_given));
    return DEER_OK;
}

static int run_proj(const deer_gru_params *p, const float *x, float *u, size_t N, cudaStream_t st)
{
    const int n3 = 3 * p->n, m = p->m;
    if (n3 <= 256 && sizeof(float) * ((size_t)m * n3 + (size_t)PROJ_PP * (m + 1)) <= 200 * 1024)
        return run_affine(x, p->W_i, p->b_i, u, N, m, n3, 0, st);
    size_t total = N * (size_t)n3;
    unsigned blocks = (unsigned)((total + 255) / 256);
    DEER_KERNEL("proj_kernel", st, proj_kernel<<<blocks, 256, 0, st>>>(x, p->W_i, p->b_i, u, N, m, n3));
    return DEER_OK;
}

template <int N> static int launch_cell_wide(CellArgs c, cudaStream_t st)
{
    using C = CellWide<N>;
    int rc;
    if ((rc = opt_in_smem((const void *)cell_wide_kernel<N>, C::SMEM)) != DEER_OK) return rc;
    const size_t total = (size_t)c.B * c.T;
    const size_t tiles = (total + C::PT - 1) / C::PT;
    const size_t per_sm = (200 * 1024) / C::SMEM;
    const size_t cap = (size_t)num_sms() * (per_sm > 4 ? 4 : per_sm);
    const unsigned blocks = (unsigned)(tiles < cap ? tiles : cap);
    DEER_KERNEL_PDL("cell_wide_kernel", false, st, cell_wide_kernel<N>, blocks, (unsigned)C::THREADS, C::SMEM, c);
    return DEER_OK;
}

// coefficient rows + rhs only (the scan builds J_t): the hidden contraction on tensor cores
// the tensor-core coefficient cell can contract the input projection itself (no u buffer, no projection pass)
static bool coef_cell_projects(int n, int m, const float *x)
{
    return (n == 32 || n == 16) && m % 8 == 0 && m >= 8 && m <= 64 && (((uintptr_t)x) & 7) == 0;
}

template <int N> static int launch_cell_coef_mma(CellArgs c, cudaStream_t st)
{
    const bool proj = c.u == nullptr;
    const size_t SM = sizeof(float) * (2 * (size_t)N * (3 * N + 4) + 6 * N + (proj ? 2 * (size_t)c.m * (3 * N + 4) : 0));
    int rc;
    const size_t total = (size_t)c.B * c.T;
    const size_t tiles = (total + 127) / 128;
    const size_t cap = (size_t)num_sms() * 2;          // (the kernel's launch bounds: two CTAs per SM; one wave, the weights split once per CTA)
    const unsigned blocks = (unsigned)(tiles < cap ? tiles : cap);
    if (proj) {
        if ((rc = opt_in_smem((const void *)cell_coef_mma_kernel<N, true>, SM)) != DEER_OK) return rc;
        DEER_KERNEL_PDL("cell_coef_mma_kernel", false, st, (cell_coef_mma_kernel<N, true>), blocks, 256u, SM, c);
    } else {
        if ((rc = opt_in_smem((const void *)cell_coef_mma_kernel<N, false>, SM)) != DEER_OK) return rc;
        DEER_KERNEL_PDL("cell_coef_mma_kernel", false, st, (cell_coef_mma_kernel<N, false>), blocks, 256u, SM, c);
    }
    return DEER_OK;
}

template <int N> static int launch_cell_small(CellArgs c, cudaStream_t st)
{
    const size_t total = (size_t)c.B * c.T;
    const size_t epb = 256 / N;
    size_t blocks = (total + epb - 1) / epb;
    // three CTAs are resident per SM (registers): a small problem runs as one persistent wave, a large one
    // is split finer so that the last wave is balanced (measured: 21.4 vs 23.5 us on config 2; 6.4 vs 7.9 ms at T = 1e6)
    const size_t resident = (size_t)num_sms() * 3;
    const size_t cap = blocks < 16 * resident ? resident : (size_t)num_sms() * 8;
    if (blocks > cap) blocks = cap;
    const unsigned gb = (unsigned)blocks;
    if (c.u) { DEER_KERNEL_PDL("cell_small_kernel", true, st, (cell_small_kernel<N, 0>), gb, 256u, 0, c); return DEER_OK; }
    switch (c.m) {
    case 1: DEER_KERNEL_PDL("cell_small_kernel", true, st, (cell_small_kernel<N, 1>), gb, 256u, 0, c); break;
    case 2: DEER_KERNEL_PDL("cell_small_kernel", true, st, (cell_small_kernel<N, 2>), gb, 256u, 0, c); break;
    case 4: DEER_KERNEL_PDL("cell_small_kernel", true, st, (cell_small_kernel<N, 4>), gb, 256u, 0, c); break;
    case 8: DEER_KERNEL_PDL("cell_small_kernel", true, st, (cell_small_kernel<N, 8>), gb, 256u, 0, c); break;
    default: return DEER_ERR_INVALID_ARG;
    }
    return DEER_OK;
}

// the cell kernel can project x itself (no u buffer, no proj pass) for these sizes
static bool cell_projects(int n, int m)
{
    return (n == 1 || n == 2 || n == 4 || n == 8) && (m == 1 || m == 2 || m == 4 || m == 8);
}

static int run_cell(CellArgs c, cudaStream_t st, bool generic = false)
{
    const bool aligned = (((uintptr_t)c.y | (uintptr_t)c.y0 | (uintptr_t)c.J) & 15) == 0;
    if (aligned && !generic) {
        switch (c.n) {
        case 1: return launch_cell_small<1>(c, st);
        case 2: return launch_cell_small<2>(c, st);
        case 4: return launch_cell_small<4>(c, st);
        case 8: return launch_cell_small<8>(c, st);
        default: break;
        }
        if ((c.u || (c.coef_only && c.residual && coef_cell_projects(c.n, c.m, c.x))) && (((uintptr_t)c.W_h) & 15) == 0) {
            switch (c.n) {
            case 16: return (c.coef_only && !c.u) ? launch_cell_coef_mma<16>(c, st) : launch_cell_wide<16>(c, st);
            case 32: return c.coef_only ? launch_cell_coef_mma<32>(c, st) : launch_cell_wide<32>(c, st);
            case 64: return (c.coef_only && c.u) ? launch_cell_coef_mma<64>(c, st) : launch_cell_wide<64>(c, st);
            default: break;
            }
        }
    }
    const int n = c.n;
    size_t sm = sizeof(float) * (3 * n * (n + 1) + 3 * n);
    int rc;
    if ((rc = opt_in_smem((const void *)cell_kernel, sm)) != DEER_OK) return rc;
    int threads = 256;
    int epb = threads / n;
    size_t N = (size_t)c.B * c.T;
    unsigned blocks = (unsigned)((N + epb - 1) / epb);
    DEER_KERNEL("cell_kernel", st, cell_kernel<<<blocks, threads, sm, st>>>(c));
    return DEER_OK;
}

template <int N> static int launch_vjp_cell_wide_n(VjpArgs v, cudaStream_t st)
{
    using C = CellWide<N>;
    const size_t sm = sizeof(float) * (3 * N * N + 3 * N + C::PT * C::HS);
    int rc;
    if ((rc = opt_in_smem((const void *)vjp_cell_wide_kernel<N>, sm)) != DEER_OK) return rc;
    const size_t total = (size_t)v.B * v.T;
    const size_t tiles = (total + C::PT - 1) / C::PT;
    const size_t per_sm = (200 * 1024) / sm;
    const size_t cap = (size_t)num_sms() * (per_sm > 4 ? 4 : per_sm);
    const unsigned blocks = (unsigned)(tiles < cap ? tiles : cap);
    DEER_KERNEL("vjp_cell_wide_kernel", st, vjp_cell_wide_kernel<N><<<blocks, C::THREADS, sm, st>>>(v));
    return DEER_OK;
}

static int launch_vjp_cell_wide(VjpArgs v, cudaStream_t st)
{
    switch (v.n) {
    case 16: return launch_vjp_cell_wide_n<16>(v, st);
    case 32: return launch_vjp_cell_wide_n<32>(v, st);
    case 64: return launch_vjp_cell_wide_n<64>(v, st);
    default: return DEER_ERR_UNSUPPORTED_N;
    }
}

static bool valid_sizes(int B, int T, int n, int m)
{
    return B > 0 && T > 0 && n > 0 && m > 0 && (double)B * T * n * n < 9.0e18;
}

static bool supported(int n, int m) { return n >= 1 && n <= 64 && m >= 1 && m <= 1024; }

// ---------------------------------------------------------------- workspace layouts
struct EvalWs {
    StatusBlock *st;
    float *trace;        // [ERR_TRACE_CAP] err after each body (device side of err_trace)
    unsigned long long *diag;   // [B] per-sequence {err bits, inverted index} of the last body
    float *u, *J, *rhs, *yalt;
    ScanWs scan;
    size_t bytes;
};

static EvalWs carve_eval(void *ws, int B, int T, int n, int m)
{
    (void)m;
    Carver cv(ws);
    EvalWs w;
    size_t N = (size_t)B * T;
    w.st = cv.take<StatusBlock>(1);
    w.trace = cv.take<float>(ERR_TRACE_CAP);
    w.diag = cv.take<unsigned long long>((size_t)B);
    w.u = cv.take<float>(N * 3 * n);
    w.J = cv.take<float>(N * n * n);
    w.rhs = cv.take<float>(N * n);
    w.yalt = cv.take<float>(N * n);
    w.scan = carve_scan(cv, B, T, n);
    w.bytes = cv.off;
    return w;
}

struct ScanOnlyWs {
    StatusBlock *st;
    ScanWs scan;
    size_t bytes;
};

static ScanOnlyWs carve_scan_only(void *ws, int B, int T, int n)
{
    Carver cv(ws);
    ScanOnlyWs w;
    w.st = cv.take<StatusBlock>(1);
    w.scan = carve_scan(cv, B, T, n);
    w.bytes = cv.off;
    return w;
}

constexpr int WGRAD_P = 592;   // slices of the position axis in the parameter-gradient reduction

struct VjpWs {
    StatusBlock *st;
    float *u, *J, *rhs, *lam, *dGi, *dGh, *partial, *partial2;
    ScanWs scan;
    size_t bytes;
};

static VjpWs carve_vjp(void *ws, int B, int T, int n, int m)
{
    Carver cv(ws);
    VjpWs w;
    size_t N = (size_t)B * T;
    w.st = cv.take<StatusBlock>(1);
    w.u = cv.take<float>(N * 3 * n);
    w.J = cv.take<float>(N * n * n);
    w.lam = cv.take<float>(N * n);
    w.dGi = cv.take<float>(N * 3 * n);
    w.dGh = cv.take<float>(N * 3 * n);
    int kmax = (m > n ? m : n) + 1;
    w.partial = cv.take<float>((size_t)WGRAD_P * 3 * n * kmax);
    w.partial2 = cv.take<float>((size_t)WGRAD_P * 3 * n * kmax);
    w.scan = carve_scan(cv, B, T, n);
    w.rhs = nullptr;
    w.bytes = cv.off;
    return w;
}

struct ClsWs {
    float *y1, *y2, *gyA, *gyB, *pool_partial, *pooled, *dlog, *gpool, *loss;
    void *inner;
    size_t inner_bytes, bytes;
};
constexpr int POOL_SEGS = 64;

static ClsWs carve_cls(void *ws, int B, int T, int n, int m, int ncls)
{
    Carver cv(ws);
    ClsWs w;
    size_t N = (size_t)B * T;
    w.y1 = cv.take<float>(N * n);
    w.y2 = cv.take<float>(N * n);
    w.gyA = cv.take<float>(N * n);
    w.gyB = cv.take<float>(N * n);
    w.pool_partial = cv.take<float>((size_t)B * POOL_SEGS * n);
    w.pooled = cv.take<float>((size_t)B * n);
    w.dlog = cv.take<float>((size_t)B * ncls);
    w.gpool = cv.take<float>((size_t)B * n);
    w.loss = cv.take<float>(64);
    int mm = m > n ? m : n;
    size_t e = carve_eval(nullptr, B, T, n, mm).bytes;
    size_t v = carve_vjp(nullptr, B, T, n, mm).bytes;
    w.inner_bytes = e > v ? e : v;
    w.inner = cv.take<char>(w.inner_bytes);
    w.bytes = cv.off;
    return w;
}

struct OdeWs {
    StatusBlock *st;
    float *J, *rhs;
    ScanWs scan;
    size_t bytes;
};

static OdeWs carve_ode(void *ws, int B, int T, int n)
{
    Carver cv(ws);
    OdeWs w;
    w.st = cv.take<StatusBlock>(1);
    w.J = cv.take<float>((size_t)B * T * n * n);
    w.rhs = cv.take<float>((size_t)B * T * n);
    w.scan = carve_scan(cv, B, T, n);
    w.bytes = cv.off;
    return w;
}

struct LstmWs {
    StatusBlock *st;
    float *trace, *u, *J, *rhs, *yalt;
    ScanWs scan;
    size_t bytes;
};

static LstmWs carve_lstm(void *ws, int B, int T, int k)
{
    Carver cv(ws);
    LstmWs w;
    const size_t N = (size_t)B * T;
    const int n = 2 * k;
    w.st = cv.take<StatusBlock>(1);
    w.trace = cv.take<float>(ERR_TRACE_CAP);
    w.u = cv.take<float>(N * 4 * k);
    w.J = cv.take<float>(N * n * n);
    w.rhs = cv.take<float>(N * n);
    w.yalt = cv.take<float>(N * n);
    w.scan = carve_scan(cv, B, T, n);
    w.bytes = cv.off;
    return w;
}

// multi-head unit: dense batches of one stride group at a time + the inner evaluation / gradient workspace
struct MhWs {
    float *xs, *y0s, *ys, *gys, *dxs, *dy0s;
    void *inner;
    size_t inner_bytes, bytes;
};

static MhWs carve_mh(void *ws, int H, const int *strides, int B, int T, int n, int m)
{
    Carver cv(ws);
    MhWs w;
    size_t maxN = 0, maxB = 0, inner = 0;
    for (int h = 0; h < H; ++h) {
        const int s = strides[h];
        const int Tp = (T + s - 1) / s;
        const size_t Bs = (size_t)B * s;
        maxN = Bs * Tp > maxN ? Bs * Tp : maxN;
        maxB = Bs > maxB ? Bs : maxB;
        const size_t e = carve_eval(nullptr, (int)Bs, Tp, n, m).bytes, v = carve_vjp(nullptr, (int)Bs, Tp, n, m).bytes;
        inner = e > inner ? e : inner;
        inner = v > inner ? v : inner;
    }
    w.xs = cv.take<float>(maxN * m);
    w.y0s = cv.take<float>(maxB * n);
    w.ys = cv.take<float>(maxN * n);
    w.gys = cv.take<float>(maxN * n);
    w.dxs = cv.take<float>(maxN * m);
    w.dy0s = cv.take<float>(maxB * n);
    w.inner_bytes = inner;
    w.inner = cv.take<char>(inner);
    w.bytes = cv.off;
    return w;
}

static int check_mh_args(const deer_gru_params *heads, const int *strides, int H, int B, int T)
{
    if (!heads || !strides || H < 1 || B <= 0 || T <= 0) return DEER_ERR_INVALID_ARG;
    for (int h = 0; h < H; ++h) {
        if (!heads[h].W_i || !heads[h].W_h || !heads[h].b_i || !heads[h].b_h) return DEER_ERR_INVALID_ARG;
        if (heads[h].n != heads[0].n || heads[h].m != heads[0].m || heads[h].n <= 0 || heads[h].m <= 0) return DEER_ERR_INVALID_ARG;
        if (strides[h] < 1 || (long long)B * strides[h] > 0x7fffffffLL) return DEER_ERR_INVALID_ARG;
    }
    if (!supported(heads[0].n, heads[0].m)) return DEER_ERR_UNSUPPORTED_N;
    if (!valid_sizes(B, T, heads[0].n, heads[0].m)) return DEER_ERR_INVALID_ARG;
    return DEER_OK;
}

static unsigned mh_blocks(size_t total);

// strided view -> dense batch and back (128-bit moves when the layout allows)
static int mh_pack(const float *src, float *dst, int B, int T, int s, int Tp, int C, int C_src, int off, cudaStream_t st)
{
    const size_t total = (size_t)B * s * Tp * C;
    const bool v4 = C % 4 == 0 && C_src % 4 == 0 && off % 4 == 0 && ((((uintptr_t)src | (uintptr_t)dst) & 15) == 0);
    if (v4) { DEER_KERNEL("mh_pack_kernel", st, mh_pack_kernel<4><<<mh_blocks(total / 4), 256, 0, st>>>(src, dst, B, T, s, Tp, C, C_src, off)); }
    else { DEER_KERNEL("mh_pack_kernel", st, mh_pack_kernel<1><<<mh_blocks(total), 256, 0, st>>>(src, dst, B, T, s, Tp, C, C_src, off)); }
    return DEER_OK;
}

static int mh_unpack(const float *src, float *dst, int B, int T, int s, int Tp, int C, int C_dst, int off, int accumulate,
                     cudaStream_t st)
{
    const size_t total = (size_t)B * s * Tp * C;
    const bool v4 = C % 4 == 0 && C_dst % 4 == 0 && off % 4 == 0 && ((((uintptr_t)src | (uintptr_t)dst) & 15) == 0);
    if (v4) { DEER_KERNEL("mh_unpack_kernel", st, mh_unpack_kernel<4><<<mh_blocks(total / 4), 256, 0, st>>>(src, dst, B, T, s, Tp, C, C_dst, off, accumulate)); }
    else { DEER_KERNEL("mh_unpack_kernel", st, mh_unpack_kernel<1><<<mh_blocks(total), 256, 0, st>>>(src, dst, B, T, s, Tp, C, C_dst, off, accumulate)); }
    return DEER_OK;
}

static unsigned mh_blocks(size_t total)
{
    size_t b = (total + 255) / 256;
    const size_t cap = (size_t)num_sms() * 8;
    if (b > cap) b = cap;
    return (unsigned)(b < 1 ? 1 : b);
}

static int check_ws(void *ws, size_t have, size_t need)
{
    if (!ws || ((uintptr_t)ws & 255) != 0 || have < need) return DEER_ERR_WORKSPACE;
    return DEER_OK;
}

// ---------------------------------------------------------------- implementation bodies
static int linrec_scan_impl(const float *J, const float *b, const float *y0, int B, int T, int n,
                            int reverse, float *y, void *ws, size_t ws_bytes, int flags,
                            cudaStream_t st)
{
    ScanOnlyWs w = carve_scan_only(ws, B, T, n);
    int rc = check_ws(ws, ws_bytes, w.bytes);
    if (rc != DEER_OK) return rc;
    DEER_CHECK_CUDA(cudaMemsetAsync(w.st, 0, sizeof(StatusBlock), st), "memset status");
    ScanArgs a{};
    a.J = J; a.b = b; a.y0 = y0; a.y = y; a.yold = nullptr;
    a.B = B; a.T = T; a.n = n; a.reverse = reverse ? 1 : 0;
    a.L = w.scan.L; a.nch = w.scan.nch;
    a.carA = w.scan.carA; a.carB = w.scan.carB; a.starts = w.scan.starts;
    a.st = w.st;
    return run_scan(a, w.scan, flags, st);
}

// copy_st / copy_ev (optional): the stream the copy to y_host is enqueued on, and an event to order it behind `st`.
// y_host (optional, host memory): the result is also copied there.  The copy is enqueued behind every
// group of bodies, after a device-side selection of the buffer that holds the current iterate, so that
// an evaluation that converges within its first group costs one host synchronisation in all.
static int gru_eval_impl(const deer_gru_params *p, const float *x, const float *y0, int B, int T,
                         float tol, int max_iter, float *y, int *iters, float *err,
                         float *err_trace, void *ws, size_t ws_bytes, int flags, cudaStream_t st,
                         float *y_host = nullptr, float *err_b = nullptr, unsigned long long *err_argmax = nullptr,
                         cudaStream_t copy_st = nullptr, cudaEvent_t copy_ev = nullptr)
{
    const int n = p->n, m = p->m;
    EvalWs w = carve_eval(ws, B, T, n, m);
    int rc = check_ws(ws, ws_bytes, w.bytes);
    if (rc != DEER_OK) return rc;
    const size_t N = (size_t)B * T;
    const bool fused_proj = cell_projects(n, m) && ((((uintptr_t)y | (uintptr_t)y0) & 15) == 0);

    ScanArgs a{};
    a.J = w.J; a.b = w.rhs; a.y0 = y0; a.y = y;
    a.B = B; a.T = T; a.n = n; a.reverse = 0;
    a.L = w.scan.L; a.nch = w.scan.nch;
    a.carA = w.scan.carA; a.carB = w.scan.carB; a.starts = w.scan.starts;
    a.st = w.st;
    // With the single-pass scan the last CTA of every scan takes the loop decision and the scan
    // leaves its flag words cleared: a body is two launches (cell, scan).
    const bool single = scan_is_single_pass(a, w.scan, flags) && (((uintptr_t)w.yalt) & 15) == 0;
    // n = 16, 32: the cell writes coefficient rows and the scan generates J_t itself, unless the caller
    // asks for materialised Jacobians
    const bool gen_J = single && (n == 16 || n == 32 || (n == 64 && !(flags & DEER_FLAG_TCGEN05))) &&
                       !(flags & DEER_FLAG_MATERIALIZE) && ((((uintptr_t)y | (uintptr_t)y0 | (uintptr_t)p->W_h) & 15) == 0);
    // ... and the iteration runs in its Newton-update form: the scan solves for the update from a zero
    // entering update (its linear solve may then be approximate: single TF32 chain products)
    if (gen_J) { a.Wh = p->W_h; a.residual = 1; a.y0 = nullptr; }
    apply_test_flags(a, flags);
    {
        StatusBlock init;
        memset(&init, 0, sizeof(init));
        init.ctl_mode = single ? 1 : 0;
        init.max_iter = max_iter;
        init.tol = tol;
        init.trace = w.trace;
        // one launch: status block, zero initial guess, cleared words of the single-pass scan
        EvalBeginArgs e{};
        if (!(flags & DEER_FLAG_WARM_START)) { e.y = y; e.ny = N * n; }
        if (single) {
            const OnePassWs &op = w.scan.op;
            const size_t tiles = (size_t)B * op.nch;
            e.flags = op.flags; e.nflags = tiles;
            e.starts = op.starts; e.nstarts = tiles * (size_t)n;
            if (onepass_ll_aggs(n)) { e.agg_words = (unsigned long long *)op.aggs; e.nagg_words = tiles * (size_t)(n * n + n); }
        }
        const size_t words = e.ny / 4 + e.nflags + e.nstarts + e.nagg_words;
        unsigned blocks = (unsigned)((words + 1023) / 1024);
        const unsigned cap = 4u * (unsigned)num_sms();
        if (blocks > cap) blocks = cap;
        if (blocks < 1u) blocks = 1u;
        DEER_KERNEL("eval_begin_kernel", st, eval_begin_kernel<<<blocks, 256, 0, st>>>(w.st, init, e));
    }
    const bool cell_proj = gen_J && coef_cell_projects(n, m, x);     // (n = 32: the coefficient cell contracts x W_i^T itself)
    if (!fused_proj && !cell_proj && (rc = run_proj(p, x, w.u, N, st)) != DEER_OK) return rc;

    // Newton loop (App. B.1): bodies are enqueued ahead of the convergence test -- the decision at
    // the end of each body is taken on the device, and the kernels of bodies past the end return
    // at once -- so the host only synchronises once per group of bodies.
    float *buf[2] = {y, w.yalt};
    int enq = 0, group = 4;
    StatusBlock hs;
    for (;;) {
        int todo = max_iter - enq;
        if (todo > group) todo = group;
        for (int j = 0; j < todo; ++j, ++enq) {
            float *cur = buf[enq & 1], *nxt = buf[(enq + 1) & 1];
            CellArgs c{p->W_h, p->b_h, (fused_proj || cell_proj) ? nullptr : w.u, x, p->W_i, p->b_i, m, cur, y0, w.J, w.rhs, B, T, n, w.st,
                       gen_J ? 1 : 0, gen_J ? 1 : 0};
            if ((rc = run_cell(c, st)) != DEER_OK) return rc;
            a.y = nxt; a.yold = cur;
            if (single) {
                if ((rc = scan_onepass(a, w.scan.op, false, flags, st)) != DEER_OK) return rc;
            } else {
                if ((rc = scan_generic(a, st)) != DEER_OK) return rc;
                DEER_KERNEL("newton_control_kernel", st, newton_control_kernel<<<1, 1, 0, st>>>(w.st, tol, max_iter, w.trace));
            }
        }
        if (y_host) {
            size_t words = N * n / 4;
            unsigned blocks = (unsigned)((words + 1023) / 1024);
            const unsigned cap = 4u * (unsigned)num_sms();
            if (blocks > cap) blocks = cap;
            if (blocks < 1u) blocks = 1u;
            DEER_KERNEL("result_select_kernel", st, result_select_kernel<<<blocks, 256, 0, st>>>(w.st, y, w.yalt, N * n));
            if (copy_st) {      // the result leaves on a stream of its own, behind the selection
                DEER_CHECK_CUDA(cudaEventRecord(copy_ev, st), "record result event");
                DEER_CHECK_CUDA(cudaStreamWaitEvent(copy_st, copy_ev, 0), "wait result event");
            }
            DEER_CHECK_CUDA(cudaMemcpyAsync(y_host, y, N * n * sizeof(float), cudaMemcpyDeviceToHost, copy_st ? copy_st : st),
                            "copy result to host");
        }
        DEER_CHECK_CUDA(cudaMemcpyAsync(&hs, w.st, 32, cudaMemcpyDeviceToHost, st), "read status");
        DEER_CHECK_CUDA(cudaStreamSynchronize(st), "sync");
        if (hs.flags & FLAG_TIMEOUT) return DEER_ERR_DEVICE_TIMEOUT;
        if (hs.done || enq >= max_iter) break;
        group = 2;
    }
    const int k = hs.iters;
    float e;
    memcpy(&e, &hs.err_last_bits, sizeof(float));
    if ((err_b || err_argmax) && k > 0) {
        // the last two iterates are still in the two buffers (before the result copy below)
        std::vector<unsigned long long> keys((size_t)B);
        DEER_KERNEL("err_diag_kernel", st, err_diag_kernel<<<(unsigned)B, 256, 0, st>>>(buf[k & 1], buf[(k + 1) & 1], (size_t)T * n, w.diag));
        DEER_CHECK_CUDA(cudaMemcpyAsync(keys.data(), w.diag, sizeof(unsigned long long) * (size_t)B, cudaMemcpyDeviceToHost, st), "read diagnostics");
        DEER_CHECK_CUDA(cudaStreamSynchronize(st), "sync");
        unsigned long long best = 0ull;
        int best_b = 0;
        for (int b = 0; b < B; ++b) {
            const unsigned bits = (unsigned)(keys[b] >> 32);
            if (err_b) memcpy(&err_b[b], &bits, sizeof(float));
            if ((keys[b] >> 32) > (best >> 32) || b == 0) { best = keys[b]; best_b = b; }
        }
        if (err_argmax)
            *err_argmax = (unsigned long long)best_b * (unsigned long long)T * (unsigned long long)n +
                          (unsigned long long)(0xffffffffu - (unsigned)(best & 0xffffffffull));
    }
    if ((k & 1) && !y_host)
        DEER_CHECK_CUDA(cudaMemcpyAsync(y, w.yalt, N * n * sizeof(float), cudaMemcpyDeviceToDevice, st), "copy result");
    if (err_trace && k > 0)
        DEER_CHECK_CUDA(cudaMemcpyAsync(err_trace, w.trace, sizeof(float) * (size_t)(k < ERR_TRACE_CAP ? k : ERR_TRACE_CAP),
                                        cudaMemcpyDeviceToHost, st), "read trace");
    DEER_CHECK_CUDA(cudaStreamSynchronize(st), "sync");
    int status = DEER_OK;
    if (!isfinite(e)) status = DEER_NONFINITE;
    else if (e > tol && !(tol < 0.0f)) status = DEER_NOT_CONVERGED;
    if (iters) *iters = k;
    if (err) *err = e;
    return status;
}

// cell VJP, parameter-gradient slices and dx in one pass (n, m in {1,2,4,8}); P = slices written
template <int N, int M>
static int launch_vjp_small_nm(const VjpSmallArgs &v, int *P, cudaStream_t st)
{
    constexpr int EPB = 256 / N;
    constexpr size_t SM = sizeof(float) * 256 * (3 * (M + 1) + 3 * (N + 1) + 1);
    int rc = opt_in_smem((const void *)vjp_small_kernel<N, M>, SM);
    if (rc != DEER_OK) return rc;
    const size_t total = (size_t)v.B * v.T;
    size_t blocks = (total + EPB - 1) / EPB;
    if (blocks > (size_t)WGRAD_P) blocks = WGRAD_P;
    *P = (int)blocks;
    DEER_KERNEL("vjp_small_kernel", st, (vjp_small_kernel<N, M><<<(unsigned)blocks, 256, SM, st>>>(v)));
    return DEER_OK;
}

template <int N>
static int launch_vjp_small_n(const VjpSmallArgs &v, int m, int *P, cudaStream_t st)
{
    switch (m) {
    case 1: return launch_vjp_small_nm<N, 1>(v, P, st);
    case 2: return launch_vjp_small_nm<N, 2>(v, P, st);
    case 4: return launch_vjp_small_nm<N, 4>(v, P, st);
    case 8: return launch_vjp_small_nm<N, 8>(v, P, st);
    default: return DEER_ERR_UNSUPPORTED_N;
    }
}

static int launch_vjp_small(const VjpSmallArgs &v, int n, int m, int *P, cudaStream_t st)
{
    switch (n) {
    case 1: return launch_vjp_small_n<1>(v, m, P, st);
    case 2: return launch_vjp_small_n<2>(v, m, P, st);
    case 4: return launch_vjp_small_n<4>(v, m, P, st);
    case 8: return launch_vjp_small_n<8>(v, m, P, st);
    default: return DEER_ERR_UNSUPPORTED_N;
    }
}

static int gru_vjp_impl(const deer_gru_params *p, const float *x, const float *y0, const float *y,
                        const float *gy, int B, int T, const deer_gru_grads *g, float *dx,
                        float *dy0, void *ws, size_t ws_bytes, int flags, cudaStream_t st)
{
    const int n = p->n, m = p->m, n3 = 3 * n;
    VjpWs w = carve_vjp(ws, B, T, n, m);
    int rc = check_ws(ws, ws_bytes, w.bytes);
    if (rc != DEER_OK) return rc;
    const size_t N = (size_t)B * T;
    DEER_CHECK_CUDA(cudaMemsetAsync(w.st, 0, sizeof(StatusBlock), st), "memset status");
    // small n and m: the cell projects x itself and one kernel does the cell VJP, the slices of the
    // parameter-gradient reduction and dx (no u, dG_i, dG_h arrays)
    const bool small = cell_projects(n, m) && !(flags & DEER_FLAG_GENERIC) && y0 != nullptr &&
                       ((((uintptr_t)y | (uintptr_t)y0) & 15) == 0);
    if (!small && (rc = run_proj(p, x, w.u, N, st)) != DEER_OK) return rc;
    ScanArgs a{};
    a.J = w.J; a.b = gy; a.y0 = nullptr; a.y = w.lam; a.yold = nullptr;
    a.B = B; a.T = T; a.n = n; a.reverse = 1;
    a.L = w.scan.L; a.nch = w.scan.nch;
    a.carA = w.scan.carA; a.carB = w.scan.carB; a.starts = w.scan.starts;
    a.st = w.st;
    // n = 16, 32: coefficient rows instead of Jacobians, J_{t+1}^T built in the reverse scan (as in the evaluation)
    const bool gen_J = (n == 16 || n == 32) && !(flags & DEER_FLAG_MATERIALIZE) && scan_is_single_pass(a, w.scan, flags) &&
                       ((((uintptr_t)y | (uintptr_t)y0 | (uintptr_t)p->W_h) & 15) == 0);
    if (gen_J) a.Wh = p->W_h;
    CellArgs c{p->W_h, p->b_h, small ? nullptr : w.u, x, p->W_i, p->b_i, m, y, y0, w.J, nullptr, B, T, n, nullptr,
               gen_J ? 1 : 0};
    if ((rc = run_cell(c, st)) != DEER_OK) return rc;
    if ((rc = run_scan(a, w.scan, flags, st)) != DEER_OK) return rc;

    if (small) {
        VjpSmallArgs v{p->W_h, p->b_h, p->W_i, p->b_i, x, y, y0, w.lam, dx, w.partial, w.partial2, B, T};
        int P = 0;
        if ((rc = launch_vjp_small(v, n, m, &P, st)) != DEER_OK) return rc;
        DEER_KERNEL("wgrad_final_kernel", st, wgrad_final_kernel<<<(n3 * (m + 1) + 7) / 8, 256, 0, st>>>(w.partial, P, n3, m, g->dW_i, g->db_i));
        DEER_KERNEL("wgrad_final_kernel", st, wgrad_final_kernel<<<(n3 * (n + 1) + 7) / 8, 256, 0, st>>>(w.partial2, P, n3, n, g->dW_h, g->db_h));
        if (dy0) {
            DEER_KERNEL("vjp_dy0_kernel", st, vjp_dy0_kernel<<<(B * n + 127) / 128, 128, 0, st>>>(w.J, w.lam, dy0, B, T, n));
        }
        return DEER_OK;
    }
    {
        VjpArgs v{p->W_h, p->b_h, w.u, y, y0, w.lam, w.dGi, w.dGh, B, T, n};
        const bool aligned = (((uintptr_t)y | (uintptr_t)y0) & 15) == 0;
        if (aligned && (n == 16 || n == 32 || n == 64)) {
            if ((rc = launch_vjp_cell_wide(v, st)) != DEER_OK) return rc;
        } else {
            size_t sm = sizeof(float) * (3 * n * (n + 1) + 3 * n);
            if ((rc = opt_in_smem((const void *)vjp_cell_kernel, sm)) != DEER_OK) return rc;
            int epb = 256 / n;
            unsigned blocks = (unsigned)((N + epb - 1) / epb);
            DEER_KERNEL("vjp_cell_kernel", st, vjp_cell_kernel<<<blocks, 256, sm, st>>>(v));
        }
    }
    const int P = (int)(N < (size_t)WGRAD_P ? N : (size_t)WGRAD_P);
    for (int side = 0; side < 2; ++side) {
        WgradArgs wa{};
        wa.dG = side == 0 ? w.dGi : w.dGh;
        wa.V = side == 0 ? x : y;
        wa.y0 = y0;
        wa.shifted = side;
        wa.T = T; wa.n3 = n3; wa.K = side == 0 ? m : n;
        wa.N = N; wa.slice = (N + P - 1) / P;
        wa.partial = w.partial;
        int outs = n3 * (wa.K + 1);
        if (n3 <= 32 && wa.K <= 8) {
            DEER_KERNEL("wgrad_small_kernel", st, wgrad_small_kernel<<<P, 256, 0, st>>>(wa));
        } else if (n3 <= 192) {
            const bool aligned16 = ((((uintptr_t)wa.dG | (uintptr_t)wa.V | (uintptr_t)wa.y0) & 15) == 0) && n3 % 4 == 0 && wa.K % 4 == 0;
            if (aligned16) {
                const size_t sm = wgrad_staged_smem(n3);
                if ((rc = opt_in_smem((const void *)wgrad_mma_staged_kernel, sm)) != DEER_OK) return rc;
                DEER_KERNEL("wgrad_mma_kernel", st, wgrad_mma_staged_kernel<<<dim3(P, (wa.K + 63) / 64), 32 * ((n3 + 15) / 16), sm, st>>>(wa));
            } else {
                DEER_KERNEL("wgrad_mma_kernel", st, wgrad_mma_kernel<<<dim3(P, (wa.K + 63) / 64), 32 * ((n3 + 15) / 16), 0, st>>>(wa));
            }
        } else {
            int tile = 32;
            while (tile > 1 && sizeof(float) * tile * (size_t)(n3 + wa.K + 1) > 160 * 1024) tile >>= 1;
            wa.tile = tile;
            size_t sm = sizeof(float) * tile * (size_t)(n3 + wa.K + 1);
            if ((rc = opt_in_smem((const void *)wgrad_partial_kernel, sm)) != DEER_OK) return rc;
            dim3 grid(P, (outs + 255) / 256);
            DEER_KERNEL("wgrad_partial_kernel", st, wgrad_partial_kernel<<<grid, 256, sm, st>>>(wa));
        }
        DEER_KERNEL("wgrad_final_kernel", st, wgrad_final_kernel<<<(outs + 7) / 8, 256, 0, st>>>(w.partial, P, n3, wa.K,
                                                                side == 0 ? g->dW_i : g->dW_h,
                                                                side == 0 ? g->db_i : g->db_h));
    }
    if (dx) {
        if (m >= 32 && m <= 256) {
            if ((rc = run_affine(w.dGi, p->W_i, nullptr, dx, N, n3, m, 1, st)) != DEER_OK) return rc;
        } else {
            size_t total = N * (size_t)m;
            DEER_KERNEL("vjp_dx_kernel", st, vjp_dx_kernel<<<(unsigned)((total + 255) / 256), 256, 0, st>>>(w.dGi, p->W_i, dx, N, m, n3));
        }
    }
    if (dy0) {
        if (gen_J) {
            DEER_KERNEL("vjp_dy0_coef_kernel", st, vjp_dy0_coef_kernel<<<(B * n + 127) / 128, 128, 0, st>>>(w.J, p->W_h, w.lam, dy0, B, T, n));
        } else {
            DEER_KERNEL("vjp_dy0_kernel", st, vjp_dy0_kernel<<<(B * n + 127) / 128, 128, 0, st>>>(w.J, w.lam, dy0, B, T, n));
        }
    }
    return DEER_OK;
}

// ---------------------------------------------------------------- built-in scratch (no-alloc entry point)
// In host code `g_noalloc_scratch` is only a handle for the runtime, not a device address: the
// address a kernel can use comes from cudaGetSymbolAddress, looked up once per device.
static __device__ __align__(256) unsigned char g_noalloc_scratch[DEER_NOALLOC_SCRATCH_BYTES];

static std::mutex g_noalloc_mu;
static void *g_noalloc_ptr[64] = {nullptr};

static int noalloc_scratch_for_current_device(void **out)
{
    int dev = -1;
    DEER_CHECK_CUDA(cudaGetDevice(&dev), "cudaGetDevice");
    if (dev < 0 || dev >= 64) { snprintf(t_err, sizeof(t_err), "device index %d out of range", dev); return DEER_ERR_CUDA; }
    std::lock_guard<std::mutex> lk(g_noalloc_mu);
    if (!g_noalloc_ptr[dev]) {
        void *p = nullptr;
        DEER_CHECK_CUDA(cudaGetSymbolAddress(&p, g_noalloc_scratch), "cudaGetSymbolAddress(scratch)");
        if (!p || ((uintptr_t)p & 255) != 0) { snprintf(t_err, sizeof(t_err), "built-in scratch misaligned"); return DEER_ERR_CUDA; }
        g_noalloc_ptr[dev] = p;
    }
    *out = g_noalloc_ptr[dev];
    return DEER_OK;
}

}  // namespace deer

using namespace deer;

// ---------------------------------------------------------------- exported C ABI
extern "C" {

size_t deer_workspace_bytes(int op, int B, int T, int n, int m, int flags)
{
    (void)flags;
    if (op == DEER_OP_SCAN || op == DEER_OP_ODE) m = 1;
    if (!valid_sizes(B, T, n, m) || !supported(n, m)) return 0;
    switch (op) {
    case DEER_OP_EVAL: return carve_eval(nullptr, B, T, n, m).bytes;
    case DEER_OP_SCAN: return carve_scan_only(nullptr, B, T, n).bytes;
    case DEER_OP_VJP: return carve_vjp(nullptr, B, T, n, m).bytes;
    case DEER_OP_CLASSIFIER: return carve_cls(nullptr, B, T, n, m, 64).bytes;
    case DEER_OP_ODE: return n <= ODE_MAX_N ? carve_ode(nullptr, B, T, n).bytes : 0;
    case DEER_OP_LSTM: return supported(2 * n, m) ? carve_lstm(nullptr, B, T, n).bytes : 0;
    default: return 0;
    }
}

int deer_linrec_scan(const float *J, const float *b, const float *y0, int B, int T, int n,
                     int reverse, float *y, void *ws, size_t ws_bytes, int flags, void *stream)
{
    if (!J || !b || !y || B <= 0 || T <= 0 || n <= 0) return DEER_ERR_INVALID_ARG;
    if (!supported(n, 1)) return DEER_ERR_UNSUPPORTED_N;
    if (!valid_sizes(B, T, n, 1)) return DEER_ERR_INVALID_ARG;
    return linrec_scan_impl(J, b, y0, B, T, n, reverse, y, ws, ws_bytes, flags, (cudaStream_t)stream);
}

int deer_gru_eval(const deer_gru_params *p, const float *x, const float *y0, int B, int T, float tol,
                  int max_iter, float *y, int *iters, float *err, float *err_trace, void *ws,
                  size_t ws_bytes, int flags, void *stream)
{
    if (!p || !x || !y0 || !y || !p->W_i || !p->W_h || !p->b_i || !p->b_h) return DEER_ERR_INVALID_ARG;
    if (B <= 0 || T <= 0 || p->n <= 0 || p->m <= 0 || max_iter < 1 || tol != tol) return DEER_ERR_INVALID_ARG;
    if (!supported(p->n, p->m)) return DEER_ERR_UNSUPPORTED_N;
    if (!valid_sizes(B, T, p->n, p->m)) return DEER_ERR_INVALID_ARG;
    return gru_eval_impl(p, x, y0, B, T, tol, max_iter, y, iters, err, err_trace, ws, ws_bytes, flags,
                         (cudaStream_t)stream);
}

int deer_gru_eval_diag(const deer_gru_params *p, const float *x, const float *y0, int B, int T, float tol,
                       int max_iter, float *y, int *iters, float *err, float *err_trace, float *err_b,
                       unsigned long long *err_argmax, void *ws, size_t ws_bytes, int flags, void *stream)
{
    if (!p || !x || !y0 || !y || !p->W_i || !p->W_h || !p->b_i || !p->b_h) return DEER_ERR_INVALID_ARG;
    if (B <= 0 || T <= 0 || p->n <= 0 || p->m <= 0 || max_iter < 1 || tol != tol) return DEER_ERR_INVALID_ARG;
    if (!supported(p->n, p->m)) return DEER_ERR_UNSUPPORTED_N;
    if (!valid_sizes(B, T, p->n, p->m)) return DEER_ERR_INVALID_ARG;
    if ((unsigned long long)T * (unsigned long long)p->n > 0xffffffffull) return DEER_ERR_INVALID_ARG;
    return gru_eval_impl(p, x, y0, B, T, tol, max_iter, y, iters, err, err_trace, ws, ws_bytes, flags,
                         (cudaStream_t)stream, nullptr, err_b, err_argmax);
}

// Copy streams and events of the pipelined host call, one set per device, made on first use.
struct HostPipe {
    cudaStream_t h2d = nullptr, d2h = nullptr;
    cudaEvent_t ev_in = nullptr, ev_sel = nullptr, ev_out = nullptr, ev_chunk[DEER_HOST_MAX_CHUNKS] = {};
    bool ready = false;
    std::mutex mu;
};
static HostPipe g_host_pipe[MAX_DEVICES];

static int host_pipe_for_current_device(HostPipe **out)
{
    int dev = 0;
    DEER_CHECK_CUDA(cudaGetDevice(&dev), "cudaGetDevice");
    if (dev < 0 || dev >= MAX_DEVICES) return DEER_ERR_INVALID_ARG;
    HostPipe &hp = g_host_pipe[dev];
    if (!hp.ready) {
        DEER_CHECK_CUDA(cudaStreamCreateWithFlags(&hp.h2d, cudaStreamNonBlocking), "create copy stream");
        DEER_CHECK_CUDA(cudaStreamCreateWithFlags(&hp.d2h, cudaStreamNonBlocking), "create copy stream");
        DEER_CHECK_CUDA(cudaEventCreateWithFlags(&hp.ev_in, cudaEventDisableTiming), "create event");
        DEER_CHECK_CUDA(cudaEventCreateWithFlags(&hp.ev_sel, cudaEventDisableTiming), "create event");
        DEER_CHECK_CUDA(cudaEventCreateWithFlags(&hp.ev_out, cudaEventDisableTiming), "create event");
        for (int c = 0; c < DEER_HOST_MAX_CHUNKS; ++c)
            DEER_CHECK_CUDA(cudaEventCreateWithFlags(&hp.ev_chunk[c], cudaEventDisableTiming), "create event");
        hp.ready = true;
    }
    *out = &hp;
    return DEER_OK;
}

int deer_gru_eval_host_chunks(int B, int T, int *first)
{
    if (B <= 0 || T <= 0) return 0;
    // chunks of about 2^19 positions: long enough to fill the GPU, short enough that the first copy in and the last
    // copy out (the two that nothing hides) are a small part of the call (config 3: three chunks measured best of 1 ... 8)
    const long long N = (long long)B * T;
    long long nc = (N + 262144) / 524288;
    if (nc > DEER_HOST_MAX_CHUNKS) nc = DEER_HOST_MAX_CHUNKS;
    if (nc > B) nc = B;
    if (nc < 1) nc = 1;
    if (first) {
        first[0] = 0;
        for (int k = 1; k < (int)nc; ++k) {
            // equal chunks for two; from three on the first and the last weigh half: their copies are the exposed ones
            // (config 3: 4, 8, 4 sequences measured 9.1 ms per call against 9.65 for 6, 6, 4)
            long long b = nc < 3 ? ((long long)B * k + nc - 1) / nc
                                 : ((long long)B * (2 * k - 1) + (nc - 1)) / (2 * (nc - 1));
            const long long lo = first[k - 1] + 1, hi = B - (nc - k);
            first[k] = (int)(b < lo ? lo : b > hi ? hi : b);
        }
        first[nc] = B;
    }
    return (int)nc;
}

int deer_gru_eval_host_chunk(int B, int T)
{
    int first[DEER_HOST_MAX_CHUNKS + 1];
    const int nc = deer_gru_eval_host_chunks(B, T, first);
    int big = 0;
    for (int c = 0; c < nc; ++c) big = std::max(big, first[c + 1] - first[c]);
    return big;
}

int deer_gru_eval_host(const deer_gru_params *p, const float *x_host, const float *y0, int B, int T, float tol,
                       int max_iter, float *y_host, int *iters, float *err, float *x_dev, float *y_dev,
                       void *ws, size_t ws_bytes, int flags, void *stream)
{
    if (!p || !x_host || !y0 || !y_host || !x_dev || !y_dev || !p->W_i || !p->W_h || !p->b_i || !p->b_h)
        return DEER_ERR_INVALID_ARG;
    if (B <= 0 || T <= 0 || p->n <= 0 || p->m <= 0 || max_iter < 1 || tol != tol) return DEER_ERR_INVALID_ARG;
    if (!supported(p->n, p->m)) return DEER_ERR_UNSUPPORTED_N;
    if (!valid_sizes(B, T, p->n, p->m)) return DEER_ERR_INVALID_ARG;
    cudaStream_t st = (cudaStream_t)stream;
    int bnd[DEER_HOST_MAX_CHUNKS + 1];
    const int nc = deer_gru_eval_host_chunks(B, T, bnd);
    if (nc <= 1) {
        DEER_CHECK_CUDA(cudaMemcpyAsync(x_dev, x_host, sizeof(float) * (size_t)B * T * p->m, cudaMemcpyHostToDevice, st),
                        "copy x to the device");
        return gru_eval_impl(p, x_dev, y0, B, T, tol, max_iter, y_dev, iters, err, nullptr, ws, ws_bytes, flags, st, y_host);
    }
    // Sequences are independent (the batch is a map over sequences), so the batch is evaluated in chunks of sequences,
    // each with its own Newton loop: chunk c + 1 arrives and chunk c - 1 leaves while chunk c is evaluated.
    {
        EvalWs wfull = carve_eval(ws, B, T, p->n, p->m);       // (the caller sized ws for the whole batch: checked as documented)
        int rc = check_ws(ws, ws_bytes, wfull.bytes);
        if (rc != DEER_OK) return rc;
    }
    HostPipe *hp = nullptr;
    int rc = host_pipe_for_current_device(&hp);
    if (rc != DEER_OK) return rc;
    std::lock_guard<std::mutex> lk(hp->mu);
    const size_t xs = (size_t)T * p->m, ys = (size_t)T * p->n;
    DEER_CHECK_CUDA(cudaEventRecord(hp->ev_in, st), "record entry event");
    DEER_CHECK_CUDA(cudaStreamWaitEvent(hp->h2d, hp->ev_in, 0), "wait entry event");
    DEER_CHECK_CUDA(cudaStreamWaitEvent(hp->d2h, hp->ev_in, 0), "wait entry event");
    for (int c = 0; c < nc; ++c) {
        const int b0 = bnd[c], bn = bnd[c + 1] - b0;
        DEER_CHECK_CUDA(cudaMemcpyAsync(x_dev + b0 * xs, x_host + b0 * xs, sizeof(float) * bn * xs, cudaMemcpyHostToDevice, hp->h2d),
                        "copy x to the device");
        DEER_CHECK_CUDA(cudaEventRecord(hp->ev_chunk[c], hp->h2d), "record chunk event");
    }
    int status = DEER_OK, k_max = 0;
    float e_max = 0.0f;
    for (int c = 0; c < nc; ++c) {
        const int b0 = bnd[c], bn = bnd[c + 1] - b0;
        DEER_CHECK_CUDA(cudaStreamWaitEvent(st, hp->ev_chunk[c], 0), "wait chunk event");
        int k = 0;
        float e = 0.0f;
        rc = gru_eval_impl(p, x_dev + b0 * xs, y0 + (size_t)b0 * p->n, bn, T, tol, max_iter, y_dev + b0 * ys, &k, &e, nullptr,
                           ws, ws_bytes, flags, st, y_host + b0 * ys, nullptr, nullptr, hp->d2h, hp->ev_sel);
        if (rc < 0) { cudaStreamSynchronize(hp->h2d); cudaStreamSynchronize(hp->d2h); return rc; }
        if (k > k_max) k_max = k;
        if (!(e <= e_max)) e_max = e;                              // (keeps a NaN)
        if (rc == DEER_NONFINITE || (rc == DEER_NOT_CONVERGED && status == DEER_OK)) status = rc;
    }
    DEER_CHECK_CUDA(cudaEventRecord(hp->ev_out, hp->d2h), "record exit event");
    DEER_CHECK_CUDA(cudaStreamWaitEvent(st, hp->ev_out, 0), "wait exit event");
    DEER_CHECK_CUDA(cudaStreamSynchronize(hp->d2h), "sync");
    if (iters) *iters = k_max;
    if (err) *err = e_max;
    return status;
}

int deer_gru_vjp(const deer_gru_params *p, const float *x, const float *y0, const float *y,
                 const float *gy, int B, int T, const deer_gru_grads *g, float *dx, float *dy0,
                 void *ws, size_t ws_bytes, int flags, void *stream)
{
    if (!p || !x || !y0 || !y || !gy || !g || !p->W_i || !p->W_h || !p->b_i || !p->b_h)
        return DEER_ERR_INVALID_ARG;
    if (!g->dW_i || !g->dW_h || !g->db_i || !g->db_h) return DEER_ERR_INVALID_ARG;
    if (B <= 0 || T <= 0 || p->n <= 0 || p->m <= 0) return DEER_ERR_INVALID_ARG;
    if (!supported(p->n, p->m)) return DEER_ERR_UNSUPPORTED_N;
    if (!valid_sizes(B, T, p->n, p->m)) return DEER_ERR_INVALID_ARG;
    return gru_vjp_impl(p, x, y0, y, gy, B, T, g, dx, dy0, ws, ws_bytes, flags, (cudaStream_t)stream);
}

int deer_gru_classifier_step(const deer_gru_params *l1, const deer_gru_params *l2, const float *W_o,
                             const float *b_o, int ncls, const float *x, const int *labels, int B,
                             int T, float tol, int max_iter, float *loss, int *iters,
                             const deer_gru_grads *g1, const deer_gru_grads *g2, float *dW_o,
                             float *db_o, void *ws, size_t ws_bytes, int flags, void *stream)
{
    if (!l1 || !l2 || !W_o || !b_o || !x || !labels || !loss || !g1 || !g2 || !dW_o || !db_o)
        return DEER_ERR_INVALID_ARG;
    if (B <= 0 || T <= 0 || ncls < 1 || ncls > 64 || max_iter < 1 || tol != tol) return DEER_ERR_INVALID_ARG;
    if (l1->n != l2->n || l2->m != l1->n) return DEER_ERR_INVALID_ARG;
    if (!supported(l1->n, l1->m) || !supported(l2->n, l2->m)) return DEER_ERR_UNSUPPORTED_N;
    if (B * ncls > 4096 || B * l1->n > 65536) return DEER_ERR_INVALID_ARG;
    const int n = l1->n, m = l1->m;
    cudaStream_t st = (cudaStream_t)stream;
    ClsWs w = carve_cls(ws, B, T, n, m, 64);
    int rc = check_ws(ws, ws_bytes, w.bytes);
    if (rc != DEER_OK) return rc;
    const size_t N = (size_t)B * T;
    // zero initial states live at the head of gyB until the backward pass needs it
    float *zero0 = w.gyB;
    DEER_CHECK_CUDA(cudaMemsetAsync(zero0, 0, (size_t)B * n * sizeof(float), st), "memset y0");
    int it[2] = {0, 0};
    int s1 = deer_gru_eval(l1, x, zero0, B, T, tol, max_iter, w.y1, &it[0], nullptr, nullptr, w.inner,
                           w.inner_bytes, flags, stream);
    if (s1 < 0) return s1;
    int s2 = deer_gru_eval(l2, w.y1, zero0, B, T, tol, max_iter, w.y2, &it[1], nullptr, nullptr,
                           w.inner, w.inner_bytes, flags, stream);
    if (s2 < 0) return s2;
    if (iters) { iters[0] = it[0]; iters[1] = it[1]; }
    int seg_len = (T + POOL_SEGS - 1) / POOL_SEGS;
    DEER_KERNEL("pool_partial_kernel", st, pool_partial_kernel<<<dim3(POOL_SEGS, B), n, 0, st>>>(w.y2, T, n, seg_len, w.pool_partial));
    DEER_KERNEL("head_kernel", st, head_kernel<<<1, 256, 0, st>>>(w.pool_partial, POOL_SEGS, B, T, n, ncls, W_o, b_o, labels,
                                   w.pooled, w.dlog, w.gpool, dW_o, db_o, w.loss));
    size_t total = N * n;
    DEER_KERNEL("broadcast_gy_kernel", st, broadcast_gy_kernel<<<(unsigned)((total + 255) / 256), 256, 0, st>>>(w.gpool, w.gyA, total, T, n));
    // zero states again (gyB is about to be overwritten by dx of layer 2): use pooled' neighbour
    float *zero1 = w.pool_partial;   // >= B*n floats, no longer needed
    DEER_CHECK_CUDA(cudaMemsetAsync(zero1, 0, (size_t)B * n * sizeof(float), st), "memset y0");
    // the backward passes are asynchronous and share one status block: the flags word of each is
    // saved beside the loss before the next call clears it, and both are read after the final sync
    const unsigned *vflags = &reinterpret_cast<const StatusBlock *>(w.inner)->flags;
    rc = deer_gru_vjp(l2, w.y1, zero1, w.y2, w.gyA, B, T, g2, w.gyB, nullptr, w.inner, w.inner_bytes,
                      flags, stream);
    if (rc != DEER_OK) return rc;
    DEER_CHECK_CUDA(cudaMemcpyAsync(w.loss + 1, vflags, sizeof(unsigned), cudaMemcpyDeviceToDevice, st), "save status");
    rc = deer_gru_vjp(l1, x, zero1, w.y1, w.gyB, B, T, g1, nullptr, nullptr, w.inner, w.inner_bytes,
                      flags, stream);
    if (rc != DEER_OK) return rc;
    DEER_CHECK_CUDA(cudaMemcpyAsync(w.loss + 2, vflags, sizeof(unsigned), cudaMemcpyDeviceToDevice, st), "save status");
    float tail[3];
    DEER_CHECK_CUDA(cudaMemcpyAsync(tail, w.loss, sizeof(tail), cudaMemcpyDeviceToHost, st), "read loss");
    DEER_CHECK_CUDA(cudaStreamSynchronize(st), "sync");
    unsigned f1, f2;
    memcpy(&f1, &tail[1], sizeof(unsigned)); memcpy(&f2, &tail[2], sizeof(unsigned));
    if ((f1 | f2) & FLAG_TIMEOUT) return DEER_ERR_DEVICE_TIMEOUT;
    *loss = tail[0];
    return s1 > s2 ? s1 : s2;
}

int deer_gru_jvp(const deer_gru_params *p, const deer_gru_params *dp, const float *x, const float *dx, const float *y0,
                 const float *dy0, const float *y, int B, int T, float *dy, void *ws, size_t ws_bytes, int flags,
                 void *stream)
{
    if (!p || !x || !y0 || !y || !dy || !p->W_i || !p->W_h || !p->b_i || !p->b_h) return DEER_ERR_INVALID_ARG;
    if (B <= 0 || T <= 0 || p->n <= 0 || p->m <= 0) return DEER_ERR_INVALID_ARG;
    if (dp && (dp->n != p->n || dp->m != p->m)) return DEER_ERR_INVALID_ARG;
    if (!supported(p->n, p->m)) return DEER_ERR_UNSUPPORTED_N;
    if (!valid_sizes(B, T, p->n, p->m)) return DEER_ERR_INVALID_ARG;
    const int n = p->n, m = p->m, n3 = 3 * n;
    cudaStream_t st = (cudaStream_t)stream;
    // the gradient's workspace layout holds what is needed: u, J, and three [B,T,3n] / [B,T,n] arrays
    VjpWs w = carve_vjp(ws, B, T, n, m);
    int rc = check_ws(ws, ws_bytes, w.bytes);
    if (rc != DEER_OK) return rc;
    const size_t N = (size_t)B * T;
    DEER_CHECK_CUDA(cudaMemsetAsync(w.st, 0, sizeof(StatusBlock), st), "memset status");
    if ((rc = run_proj(p, x, w.u, N, st)) != DEER_OK) return rc;
    // du1 = x dW_i^T + db_i ;  du2 = dx W_i^T
    float *du1 = nullptr, *du2 = nullptr;
    const bool have_di = dp && (dp->W_i || dp->b_i);
    if (have_di) {
        if (!dp->W_i || !dp->b_i) return DEER_ERR_INVALID_ARG;       // the input-side pair comes together
        deer_gru_params q = *p;
        q.W_i = dp->W_i; q.b_i = dp->b_i;
        du1 = w.dGi;
        if ((rc = run_proj(&q, x, du1, N, st)) != DEER_OK) return rc;
    }
    if (dx) {
        du2 = w.dGh;
        if ((rc = run_affine(dx, p->W_i, nullptr, du2, N, m, n3, 0, st)) != DEER_OK) return rc;
    }
    if (dp && ((dp->W_h == nullptr) != (dp->b_h == nullptr))) return DEER_ERR_INVALID_ARG;
    {
        JvpArgs j{p->W_h, p->b_h, dp ? dp->W_h : nullptr, dp ? dp->b_h : nullptr, w.u, du1, du2, y, y0, w.lam, B, T, n};
        const size_t sm = sizeof(float) * (6 * (size_t)n * (n + 1) + 6 * n);
        if ((rc = opt_in_smem((const void *)jvp_cell_kernel, sm)) != DEER_OK) return rc;
        const int epb = 256 / n;
        size_t blocks = (N + epb - 1) / epb;
        const size_t cap = (size_t)num_sms() * 8;
        if (blocks > cap) blocks = cap;
        DEER_KERNEL("jvp_cell_kernel", st, jvp_cell_kernel<<<(unsigned)blocks, 256, sm, st>>>(j));
    }
    // the Jacobians at the trajectory (exact: a one-shot solve), then dy = L_G^{-1}[df] from dy0 (Sec. 3.1.1)
    ScanArgs a{};
    a.J = w.J; a.b = w.lam; a.y0 = dy0; a.y = dy; a.yold = nullptr;
    a.B = B; a.T = T; a.n = n; a.reverse = 0;
    a.L = w.scan.L; a.nch = w.scan.nch;
    a.carA = w.scan.carA; a.carB = w.scan.carB; a.starts = w.scan.starts;
    a.st = w.st;
    CellArgs c{p->W_h, p->b_h, w.u, x, p->W_i, p->b_i, m, y, y0, w.J, nullptr, B, T, n, nullptr, 0, 0};
    if ((rc = run_cell(c, st)) != DEER_OK) return rc;
    return run_scan(a, w.scan, flags, st);
}

int deer_lstm_eval(const deer_lstm_params *p, const float *x, const float *s0, int B, int T, float tol, int max_iter,
                   float *s_out, int *iters, float *err, void *ws, size_t ws_bytes, int flags, void *stream)
{
    if (!p || !x || !s0 || !s_out || !p->W_i || !p->W_h || !p->b) return DEER_ERR_INVALID_ARG;
    if (B <= 0 || T <= 0 || p->k <= 0 || p->m <= 0 || max_iter < 1 || tol != tol) return DEER_ERR_INVALID_ARG;
    if (!supported(2 * p->k, p->m)) return DEER_ERR_UNSUPPORTED_N;
    if (!valid_sizes(B, T, 2 * p->k, p->m)) return DEER_ERR_INVALID_ARG;
    const int k = p->k, m = p->m, n = 2 * k;
    cudaStream_t st = (cudaStream_t)stream;
    LstmWs w = carve_lstm(ws, B, T, k);
    int rc = check_ws(ws, ws_bytes, w.bytes);
    if (rc != DEER_OK) return rc;
    const size_t N = (size_t)B * T;

    ScanArgs a{};
    a.J = w.J; a.b = w.rhs; a.y0 = s0; a.y = s_out;
    a.B = B; a.T = T; a.n = n; a.reverse = 0;
    a.L = w.scan.L; a.nch = w.scan.nch;
    a.carA = w.scan.carA; a.carB = w.scan.carB; a.starts = w.scan.starts;
    a.st = w.st;
    apply_test_flags(a, flags);
    const bool single = scan_is_single_pass(a, w.scan, flags) && (((uintptr_t)w.yalt) & 15) == 0;
    {
        StatusBlock init;
        memset(&init, 0, sizeof(init));
        init.ctl_mode = single ? 1 : 0;
        init.max_iter = max_iter;
        init.tol = tol;
        init.trace = w.trace;
        EvalBeginArgs e{};
        if (!(flags & DEER_FLAG_WARM_START)) { e.y = s_out; e.ny = N * n; }
        if (single) {
            const OnePassWs &op = w.scan.op;
            const size_t tiles = (size_t)B * op.nch;
            e.flags = op.flags; e.nflags = tiles;
            e.starts = op.starts; e.nstarts = tiles * (size_t)n;
            if (onepass_ll_aggs(n)) { e.agg_words = (unsigned long long *)op.aggs; e.nagg_words = tiles * (size_t)(n * n + n); }
        }
        const size_t words = e.ny / 4 + e.nflags + e.nstarts + e.nagg_words;
        unsigned blocks = (unsigned)((words + 1023) / 1024);
        const unsigned cap = 4u * (unsigned)num_sms();
        if (blocks > cap) blocks = cap;
        if (blocks < 1u) blocks = 1u;
        DEER_KERNEL("eval_begin_kernel", st, eval_begin_kernel<<<blocks, 256, 0, st>>>(w.st, init, e));
    }
    // u = x W_i^T + b  (4k outputs per position; iteration-invariant)
    if (sizeof(float) * ((size_t)m * 4 * k + (size_t)PROJ_PP * (m + 1)) <= 200 * 1024 && 4 * k <= 256) {
        if ((rc = run_affine(x, p->W_i, p->b, w.u, N, m, 4 * k, 0, st)) != DEER_OK) return rc;
    } else {
        const size_t total = N * (size_t)(4 * k);
        DEER_KERNEL("proj_kernel", st, proj_kernel<<<(unsigned)((total + 255) / 256), 256, 0, st>>>(x, p->W_i, p->b, w.u, N, m, 4 * k));
    }
    const size_t sm = sizeof(float) * 4 * (size_t)k * (k + 1);
    if ((rc = opt_in_smem((const void *)lstm_cell_kernel, sm)) != DEER_OK) return rc;
    const int threads = 256 / k * k;
    size_t cblocks = (N + (size_t)(256 / k) - 1) / (size_t)(256 / k);
    if (cblocks > (size_t)num_sms() * 16) cblocks = (size_t)num_sms() * 16;

    float *buf[2] = {s_out, w.yalt};
    int enq = 0, group = 4;
    StatusBlock hs;
    for (;;) {
        int todo = max_iter - enq;
        if (todo > group) todo = group;
        for (int j = 0; j < todo; ++j, ++enq) {
            float *cur = buf[enq & 1], *nxt = buf[(enq + 1) & 1];
            LstmCellArgs c{p->W_h, w.u, cur, s0, w.J, w.rhs, B, T, k, w.st};
            DEER_KERNEL("lstm_cell_kernel", st, lstm_cell_kernel<<<(unsigned)cblocks, threads, sm, st>>>(c));
            a.y = nxt; a.yold = cur;
            if (single) {
                if ((rc = scan_onepass(a, w.scan.op, false, flags, st)) != DEER_OK) return rc;
            } else {
                if ((rc = scan_generic(a, st)) != DEER_OK) return rc;
                DEER_KERNEL("newton_control_kernel", st, newton_control_kernel<<<1, 1, 0, st>>>(w.st, tol, max_iter, w.trace));
            }
        }
        DEER_CHECK_CUDA(cudaMemcpyAsync(&hs, w.st, 32, cudaMemcpyDeviceToHost, st), "read status");
        DEER_CHECK_CUDA(cudaStreamSynchronize(st), "sync");
        if (hs.flags & FLAG_TIMEOUT) return DEER_ERR_DEVICE_TIMEOUT;
        if (hs.done || enq >= max_iter) break;
        group = 2;
    }
    const int kk = hs.iters;
    float e;
    memcpy(&e, &hs.err_last_bits, sizeof(float));
    if (kk & 1)
        DEER_CHECK_CUDA(cudaMemcpyAsync(s_out, w.yalt, N * n * sizeof(float), cudaMemcpyDeviceToDevice, st), "copy result");
    DEER_CHECK_CUDA(cudaStreamSynchronize(st), "sync");
    int status = DEER_OK;
    if (!isfinite(e)) status = DEER_NONFINITE;
    else if (e > tol && !(tol < 0.0f)) status = DEER_NOT_CONVERGED;
    if (iters) *iters = kk;
    if (err) *err = e;
    return status;
}

int deer_ode_linear_solve(const float *G, const float *z, const float *t, const float *y0, int B, int T, int n, float *y,
                          void *ws, size_t ws_bytes, int flags, void *stream)
{
    if (!G || !z || !t || !y0 || !y || B <= 0 || T <= 0 || n <= 0) return DEER_ERR_INVALID_ARG;
    if (n > ODE_MAX_N) return DEER_ERR_UNSUPPORTED_N;
    if (!valid_sizes(B, T, n, 1)) return DEER_ERR_INVALID_ARG;
    cudaStream_t st = (cudaStream_t)stream;
    OdeWs w = carve_ode(ws, B, T, n);
    int rc = check_ws(ws, ws_bytes, w.bytes);
    if (rc != DEER_OK) return rc;
    DEER_CHECK_CUDA(cudaMemsetAsync(w.st, 0, sizeof(StatusBlock), st), "memset status");
    {
        const size_t sm = sizeof(float) * 3 * (size_t)(n + 1) * (n + 1) * ODE_THREADS;
        if ((rc = opt_in_smem((const void *)ode_discretise_kernel, sm)) != DEER_OK) return rc;
        size_t blocks = ((size_t)B * T + ODE_THREADS - 1) / ODE_THREADS;
        const size_t cap = (size_t)num_sms() * 8;
        if (blocks > cap) blocks = cap;
        DEER_KERNEL("ode_discretise_kernel", st, ode_discretise_kernel<<<(unsigned)blocks, ODE_THREADS, sm, st>>>(G, z, t, w.J, w.rhs, B, T, n));
    }
    ScanArgs a{};
    a.J = w.J; a.b = w.rhs; a.y0 = y0; a.y = y; a.yold = nullptr;
    a.B = B; a.T = T; a.n = n; a.reverse = 0;
    a.L = w.scan.L; a.nch = w.scan.nch;
    a.carA = w.scan.carA; a.carB = w.scan.carB; a.starts = w.scan.starts;
    a.st = w.st;
    return run_scan(a, w.scan, flags, st);
}

size_t deer_multihead_workspace_bytes(const int *strides, int H, int B, int T, int n, int m, int flags)
{
    (void)flags;
    if (!strides || H < 1 || !valid_sizes(B, T, n, m) || !supported(n, m)) return 0;
    for (int h = 0; h < H; ++h)
        if (strides[h] < 1 || (long long)B * strides[h] > 0x7fffffffLL) return 0;
    return carve_mh(nullptr, H, strides, B, T, n, m).bytes;
}

// Heads in order of stride (stable): heads of equal stride read the same dense batch of x, which is then packed once.
static std::vector<int> mh_order(const int *strides, int H)
{
    std::vector<int> order((size_t)H);
    for (int h = 0; h < H; ++h) order[(size_t)h] = h;
    std::stable_sort(order.begin(), order.end(), [&](int a, int b) { return strides[a] < strides[b]; });
    return order;
}

int deer_gru_multihead_eval(const deer_gru_params *heads, const int *strides, int H, const float *x, const float *y0,
                            int B, int T, float tol, int max_iter, float *y, int *iters, void *ws, size_t ws_bytes,
                            int flags, void *stream)
{
    int rc = check_mh_args(heads, strides, H, B, T);
    if (rc != DEER_OK) return rc;
    if (!x || !y0 || !y || max_iter < 1 || tol != tol) return DEER_ERR_INVALID_ARG;
    const int n = heads[0].n, m = heads[0].m;
    cudaStream_t st = (cudaStream_t)stream;
    MhWs w = carve_mh(ws, H, strides, B, T, n, m);
    if ((rc = check_ws(ws, ws_bytes, w.bytes)) != DEER_OK) return rc;
    int worst = DEER_OK;
    int packed_stride = 1;                     // stride whose dense batch of x is in w.xs (stride 1: x itself)
    const std::vector<int> order = mh_order(strides, H);
    for (int oi = 0; oi < H; ++oi) {
        const int h = order[(size_t)oi];
        const int s = strides[h], Tp = (T + s - 1) / s, Bs = B * s;
        if (s != packed_stride) {              // heads of equal stride read the same dense batch of x
            { if ((rc = mh_pack(x, w.xs, B, T, s, Tp, m, m, 0, st)) != DEER_OK) return rc; }
            packed_stride = s;
        }
        const float *xs = s == 1 ? x : w.xs;
        DEER_KERNEL("mh_y0_pack_kernel", st, mh_y0_pack_kernel<<<mh_blocks((size_t)Bs * n), 256, 0, st>>>(y0, w.y0s, B, s, n, H, h));
        if (flags & DEER_FLAG_WARM_START)
            { if ((rc = mh_pack(y, w.ys, B, T, s, Tp, n, H * n, h * n, st)) != DEER_OK) return rc; }
        int it = 0;
        rc = gru_eval_impl(&heads[h], xs, w.y0s, Bs, Tp, tol, max_iter, w.ys, &it, nullptr, nullptr, w.inner, w.inner_bytes,
                           flags, st);
        if (rc < 0) return rc;
        if (iters) iters[h] = it;
        if (rc > worst) worst = rc;
        { if ((rc = mh_unpack(w.ys, y, B, T, s, Tp, n, H * n, h * n, 0, st)) != DEER_OK) return rc; }
    }
    DEER_CHECK_CUDA(cudaStreamSynchronize(st), "sync");
    return worst;
}

int deer_gru_multihead_vjp(const deer_gru_params *heads, const int *strides, int H, const float *x, const float *y0,
                           const float *y, const float *gy, int B, int T, const deer_gru_grads *dheads, float *dx,
                           float *dy0, void *ws, size_t ws_bytes, int flags, void *stream)
{
    int rc = check_mh_args(heads, strides, H, B, T);
    if (rc != DEER_OK) return rc;
    if (!x || !y0 || !y || !gy || !dheads) return DEER_ERR_INVALID_ARG;
    for (int h = 0; h < H; ++h)
        if (!dheads[h].dW_i || !dheads[h].dW_h || !dheads[h].db_i || !dheads[h].db_h) return DEER_ERR_INVALID_ARG;
    const int n = heads[0].n, m = heads[0].m;
    cudaStream_t st = (cudaStream_t)stream;
    MhWs w = carve_mh(ws, H, strides, B, T, n, m);
    if ((rc = check_ws(ws, ws_bytes, w.bytes)) != DEER_OK) return rc;
    unsigned timeout_flags = 0;
    int packed_stride = 1;                     // (stride 1: x itself)
    const std::vector<int> order = mh_order(strides, H);
    for (int oi = 0; oi < H; ++oi) {
        const int h = order[(size_t)oi];
        const int s = strides[h], Tp = (T + s - 1) / s, Bs = B * s;
        if (s != packed_stride) {
            { if ((rc = mh_pack(x, w.xs, B, T, s, Tp, m, m, 0, st)) != DEER_OK) return rc; }
            packed_stride = s;
        }
        const float *xs = s == 1 ? x : w.xs;
        DEER_KERNEL("mh_y0_pack_kernel", st, mh_y0_pack_kernel<<<mh_blocks((size_t)Bs * n), 256, 0, st>>>(y0, w.y0s, B, s, n, H, h));
        { if ((rc = mh_pack(y, w.ys, B, T, s, Tp, n, H * n, h * n, st)) != DEER_OK) return rc; }
        { if ((rc = mh_pack(gy, w.gys, B, T, s, Tp, n, H * n, h * n, st)) != DEER_OK) return rc; }
        rc = gru_vjp_impl(&heads[h], xs, w.y0s, w.ys, w.gys, Bs, Tp, &dheads[h], dx ? w.dxs : nullptr, dy0 ? w.dy0s : nullptr,
                          w.inner, w.inner_bytes, flags, st);
        if (rc != DEER_OK) return rc;
        if (dx)     // the heads' input gradients add up, head by head in a fixed order (that of the strides)
            { if ((rc = mh_unpack(w.dxs, dx, B, T, s, Tp, m, m, 0, oi > 0, st)) != DEER_OK) return rc; }
        if (dy0)
            DEER_KERNEL("mh_dy0_reduce_kernel", st, mh_dy0_reduce_kernel<<<mh_blocks((size_t)B * n), 256, 0, st>>>(w.dy0s, dy0, B, s, n, H, h));
        // the inner gradient calls share one status block: keep every head's flags
        unsigned f = 0;
        DEER_CHECK_CUDA(cudaMemcpyAsync(&f, &reinterpret_cast<const StatusBlock *>(w.inner)->flags, sizeof(unsigned),
                                        cudaMemcpyDeviceToHost, st), "read status");
        DEER_CHECK_CUDA(cudaStreamSynchronize(st), "sync");
        timeout_flags |= f;
    }
    return (timeout_flags & FLAG_TIMEOUT) ? DEER_ERR_DEVICE_TIMEOUT : DEER_OK;
}

int deer_linrec_scan_noalloc(const float *J, const float *b, const float *y0, int B, int T, int n,
                             int reverse, float *y, void *stream)
{
    if (!J || !b || !y || B <= 0 || T <= 0 || n <= 0) return DEER_ERR_INVALID_ARG;
    if (!supported(n, 1)) return DEER_ERR_UNSUPPORTED_N;
    if (!valid_sizes(B, T, n, 1)) return DEER_ERR_INVALID_ARG;
    const size_t need = carve_scan_only(nullptr, B, T, n).bytes;
    if (need > sizeof(g_noalloc_scratch)) {
        snprintf(t_err, sizeof(t_err),
                 "deer_linrec_scan_noalloc: B=%d T=%d n=%d needs %zu bytes of scratch, the built-in array holds %zu",
                 B, T, n, need, sizeof(g_noalloc_scratch));
        return DEER_ERR_WORKSPACE;
    }
    void *scratch = nullptr;
    int rc = noalloc_scratch_for_current_device(&scratch);
    if (rc != DEER_OK) return rc;
    // linrec_scan_impl clears what has to start at zero (status block, tile flags, entering-state
    // words, counters) with stream-ordered memsets on every call; nothing else is read before written
    return linrec_scan_impl(J, b, y0, B, T, n, reverse, y, scratch, sizeof(g_noalloc_scratch), 0,
                            (cudaStream_t)stream);
}

static int status_from_block(const void *block, cudaStream_t st)
{
    StatusBlock hs;
    DEER_CHECK_CUDA(cudaMemcpyAsync(&hs, block, 32, cudaMemcpyDeviceToHost, st), "read status");
    DEER_CHECK_CUDA(cudaStreamSynchronize(st), "sync");
    return (hs.flags & FLAG_TIMEOUT) ? DEER_ERR_DEVICE_TIMEOUT : DEER_OK;
}

int deer_workspace_status(const void *ws, void *stream)
{
    if (!ws || ((uintptr_t)ws & 255) != 0) return DEER_ERR_WORKSPACE;
    return status_from_block(ws, (cudaStream_t)stream);
}

int deer_noalloc_status(void *stream)
{
    void *scratch = nullptr;
    int rc = noalloc_scratch_for_current_device(&scratch);
    if (rc != DEER_OK) return rc;
    return status_from_block(scratch, (cudaStream_t)stream);
}

int deer_scan_geometry(int B, int T, int n, int flags, int *out)
{
    if (!out || B <= 0 || T <= 0 || n <= 0) return DEER_ERR_INVALID_ARG;
    if (!supported(n, 1)) return DEER_ERR_UNSUPPORTED_N;
    if (!valid_sizes(B, T, n, 1)) return DEER_ERR_INVALID_ARG;
    const bool umma = (flags & DEER_FLAG_TCGEN05) != 0;
    int sw = 0;
    const int L1 = onepass_tile_len(n, B, T, &sw);
    const bool single = L1 > 0 && !(flags & DEER_FLAG_GENERIC) && B <= single_pass_max_batch(n, umma);
    if (single) {
        int res_warps = 0, max_seq = 0, res_cap = 8;
        switch (n) {
        case 1: case 2: case 4: res_warps = n == 4 ? OnePass<4>::WARPS : OnePass<1>::WARPS; max_seq = OnePass<1>::MAX_SEQ_PER_WARP; break;
        case 8: res_warps = Warp8::RES_WARPS; max_seq = OnePass<8>::MAX_SEQ_PER_WARP; break;
        case 16: case 32: res_warps = big_res_warps(B); max_seq = WarpN<16>::MAX_SEQ_PER_WARP; break;
        default: res_warps = umma ? Umma64::RES_WARPS : res_warps64(B); max_seq = Cta64::MAX_SEQ_PER_WARP; res_cap = umma ? 8 : 16; break;
        }
        out[0] = 1; out[1] = L1; out[2] = sw; out[3] = (T + L1 - 1) / L1;
        out[4] = resolver_ctas(B, res_warps, max_seq, res_cap);
    } else {
        const int L = gen_chunk_len(T);
        out[0] = 0; out[1] = L; out[2] = 0; out[3] = (T + L - 1) / L; out[4] = 0;
    }
    out[5] = num_sms();
    return DEER_OK;
}

int deer_gru_cell_jac(const deer_gru_params *p, const float *x, const float *y0, const float *y, int B, int T,
                      float *J, float *rhs, void *ws, size_t ws_bytes, int flags, void *stream)
{
    if (!p || !x || !y0 || !y || !J || !rhs || !p->W_i || !p->W_h || !p->b_i || !p->b_h) return DEER_ERR_INVALID_ARG;
    if (B <= 0 || T <= 0 || p->n <= 0 || p->m <= 0) return DEER_ERR_INVALID_ARG;
    if (!supported(p->n, p->m)) return DEER_ERR_UNSUPPORTED_N;
    if (!valid_sizes(B, T, p->n, p->m)) return DEER_ERR_INVALID_ARG;
    const int n = p->n, m = p->m;
    const bool coef = (flags & DEER_FLAG_COEF_ROWS) != 0;
    if (coef && !(n == 16 || n == 32 || n == 64)) return DEER_ERR_UNSUPPORTED_N;
    if (coef && (flags & DEER_FLAG_GENERIC)) return DEER_ERR_INVALID_ARG;
    if (coef && ((((uintptr_t)y | (uintptr_t)y0 | (uintptr_t)J | (uintptr_t)p->W_h) & 15) != 0)) return DEER_ERR_INVALID_ARG;
    cudaStream_t st = (cudaStream_t)stream;
    EvalWs w = carve_eval(ws, B, T, n, m);
    int rc = check_ws(ws, ws_bytes, w.bytes);
    if (rc != DEER_OK) return rc;
    const bool generic = (flags & DEER_FLAG_GENERIC) != 0;
    const bool fused_proj = !generic && cell_projects(n, m) && ((((uintptr_t)y | (uintptr_t)y0 | (uintptr_t)J) & 15) == 0);
    if (!fused_proj && (rc = run_proj(p, x, w.u, (size_t)B * T, st)) != DEER_OK) return rc;
    CellArgs c{p->W_h, p->b_h, fused_proj ? nullptr : w.u, x, p->W_i, p->b_i, m, y, y0, J, rhs, B, T, n, nullptr, coef ? 1 : 0};
    return run_cell(c, st, generic);
}

const char *deer_status_string(int s)
{
    switch (s) {
    case DEER_OK: return "ok";
    case DEER_NOT_CONVERGED: return "not converged within max_iter";
    case DEER_NONFINITE: return "non-finite values in the iterate";
    case DEER_ERR_INVALID_ARG: return "invalid argument";
    case DEER_ERR_UNSUPPORTED_N: return "unsupported hidden or input size";
    case DEER_ERR_WORKSPACE: return "workspace missing, misaligned or too small";
    case DEER_ERR_CUDA: return "CUDA runtime error";
    case DEER_ERR_DEVICE_TIMEOUT: return "bounded device-side wait expired";
    default: return "unknown status";
    }
}

const char *deer_last_error(void) { return t_err; }

long long deer_launch_count(void) { return g_launches.load(); }

void deer_profile_enable(int on)
{
    g_prof_on.store(on != 0);
}

size_t deer_profile_read(char *buf, size_t cap)
{
    std::lock_guard<std::mutex> lk(g_prof_mu);
    std::map<std::string, std::pair<long, double>> acc;
    std::vector<std::string> order;
    for (auto &r : g_prof) {
        float ms = 0.0f;
        cudaEventSynchronize(r.e1);
        cudaEventElapsedTime(&ms, r.e0, r.e1);
        cudaEventDestroy(r.e0);
        cudaEventDestroy(r.e1);
        if (!acc.count(r.name)) order.push_back(r.name);
        acc[r.name].first += 1;
        acc[r.name].second += ms;
    }
    g_prof.clear();
    std::string out;
    char line[160];
    for (auto &k : order) {
        snprintf(line, sizeof(line), "%s %ld %.6f\n", k.c_str(), acc[k].first, acc[k].second);
        out += line;
    }
    if (buf && cap) {
        size_t c = out.size() < cap - 1 ? out.size() : cap - 1;
        memcpy(buf, out.data(), c);
        buf[c] = 0;
    }
    return out.size();
}

}  // extern "C"
