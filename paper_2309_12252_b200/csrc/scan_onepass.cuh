// Single-pass chunked scan of the linear recurrence for n in {1, 2} (and the protocol, resolver
// and helpers shared by the kernels for larger n): J and b are read from HBM once, y written once.
//
//   * One persistent kernel.  Every tile of L consecutive positions of one
//     sequence is visited twice by a worker CTA: an A item (stage the tile,
//     fold it into the tile aggregate, publish the aggregate) and, a few items
//     later, a B item (stage the tile again -- by then from L2 --, replay it
//     from its entering state, write y).  A items never wait on anything; the
//     entering states are produced by resolver warps (a few CTAs that took the
//     first role tickets) which walk each sequence's published aggregates in
//     order.  Workers therefore hold no data while a dependency is in flight.
//   * Chains.  A chain is S consecutive positions.  n <= 4: one thread per
//     chain keeps the whole running aggregate (A, beta) in registers,
//     (A, beta) <- (J_t A, J_t beta + b_t), and the chain aggregates of a warp
//     and of the CTA are combined by warp-shuffle scans.  (n >= 8 share this
//     file's protocol, resolvers and helpers; their workers are in
//     scan_warp8.cuh, scan_warpn.cuh, scan_cta64.cuh.)
//   * Staging and bank conflicts.  n <= 2: the tile is dense in shared memory,
//     brought in by one bulk copy (cp.async.bulk + mbarrier), and S is chosen
//     odd (n = 2) or S/4 odd (n = 1, four positions per 128-bit load).  n = 4:
//     every chain run is padded by 16 bytes so that the stride between the
//     chains of a warp is odd in 16-byte units, staged with per-thread
//     16-byte cp.async copies.
//   * Protocol.  Roles and tile ids are handed out by atomic counters to
//     running CTAs only, and a tile's B item depends only on A items of lower
//     ids, which their owners execute immediately after claiming: no
//     co-residency assumption is needed for progress.  Aggregates (n <= 4)
//     and entering states travel as 64-bit {value, flag} words, so reading
//     one needs a single round trip and no fence (n >= 8 publish their larger
//     aggregates with a release flag).  Every wait is bounded: on expiry the
//     kernel raises FLAG_TIMEOUT and all CTAs drain.
//   * In the B item y overwrites b in shared memory and is streamed out with
//     coalesced stores fused with the max |y - y_old| reduction.
//
// Reverse scans (the adjoint) use the same kernel with reversed indexing and
// transposed register access.
#pragma once
#include "common.cuh"

namespace deer {

template <int N> struct OnePass {
    static constexpr int LPC = (N == 8) ? 4 : 1;       // lanes per chain
    static constexpr int COLS = N / LPC;               // columns of A per lane (n = 8 path)
    static constexpr int S = (N == 8) ? 5 : (N == 4) ? 5 : (N == 2) ? 9 : 28;   // positions per chain
    static constexpr int THREADS = (N >= 4) ? 128 : 256;
    static constexpr int WARPS = THREADS / 32;
    static constexpr int CHAINS = THREADS / LPC;
    static constexpr int CPW = CHAINS / WARPS;         // chains per warp
    static constexpr int L = CHAINS * S;               // positions per tile
    static constexpr bool PADDED = N >= 4;             // run-padded layout
    static constexpr int JRUN = S * N * N + (PADDED ? 4 : 0);        // floats per chain run of J
    static constexpr int BRUN = S * N + ((N == 8) ? 4 : 0);          // floats per chain run of b / y
    static constexpr int JBUF = CHAINS * JRUN, BBUF = CHAINS * BRUN;
    static constexpr int AGG = N * N + N;              // floats of one aggregate (A row-major, then beta)
    static constexpr int Q = (N == 1) ? 3 : (N == 4) ? 1 : 2;   // pending tiles (A scheduled, B not yet) per CTA
    // with one pending tile the B item follows its own A item directly: the tile stays staged and
    // each thread keeps its chain's exclusive prefix in registers
    static constexpr bool HOLD = (Q == 1);
    // kept per pending tile: exclusive chain prefixes within the warp (not when held in registers)
    // + exclusive warp prefixes
    static constexpr int PEND = ((HOLD ? 0 : CHAINS) + WARPS) * AGG;
    static constexpr int SM_FLOATS = JBUF + BBUF + Q * PEND + WARPS * 2 * AGG + N + 4;
    static constexpr size_t SMEM = SM_FLOATS * sizeof(float) + 64 + 128;
    static constexpr int MAX_SEQ_PER_WARP = 8;         // sequences one resolver warp can serve
    static_assert(32 * AGG <= JBUF / WARPS, "resolver staging must fit the tile buffer");
    // the chains a warp reads together must fall in distinct banks: chain stride odd in 16-byte
    // units (n = 1 reads four positions per load, so S/4 must be odd)
    static_assert(N == 1 ? ((S / 4) % 2 == 1 && S % 4 == 0) : ((JRUN / 4) % 2 == 1), "chain stride");
};

struct OnePassWs {
    unsigned *flags;              // [B*nch]  1 once the tile aggregate is published (n >= 8)
    float *aggs;                  // [B*nch][n*n+n] floats (n >= 8) or {flag << 32 | float bits} words (n <= 4)
    unsigned long long *starts;   // [B*nch][n]  state entering the tile as {flag << 32 | float bits}
    int nch, Wd, nwin;            // tiles per sequence, tiles per sequence per window, windows
    unsigned total_ids;
    int resolvers;                // CTAs that take the resolver role
    int res_warps;                // warps of a resolver CTA that resolve (n = 16, 32: chosen per launch)
    int sw;                       // positions per warp chain where the kernel takes it at run time (n = 8)
    float *pfx;                   // [B*nch][chains per tile - 1][n*n+n] prefix aggregates inside each tile (n = 16, 32:
                                  // written by the reduce launch of the two-launch scan of deer_gru_eval)
};

// ---------------------------------------------------------------- small PTX helpers
__device__ __forceinline__ unsigned smem_u32(const void *p) { return (unsigned)__cvta_generic_to_shared(p); }

__device__ __forceinline__ void mbar_init(uint64_t *bar, unsigned count)
{
    asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(smem_u32(bar)), "r"(count) : "memory");
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
}

__device__ __forceinline__ void mbar_arrive_expect_tx(uint64_t *bar, unsigned bytes)
{
    asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(smem_u32(bar)), "r"(bytes) : "memory");
}

__device__ __forceinline__ bool mbar_try_wait(uint64_t *bar, unsigned parity)
{
    unsigned ok;
    asm volatile("{\n\t.reg .pred p;\n\tmbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\tselp.u32 %0, 1, 0, p;\n\t}"
                 : "=r"(ok) : "r"(smem_u32(bar)), "r"(parity) : "memory");
    return ok != 0;
}

__device__ __forceinline__ void bulk_g2s(void *dst, const void *src, unsigned bytes, uint64_t *bar)
{
    asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];"
                 ::"r"(smem_u32(dst)), "l"(src), "r"(bytes), "r"(smem_u32(bar)) : "memory");
}

// 16-byte asynchronous copy global -> shared (per thread; bypasses L1)
__device__ __forceinline__ void cp_async16(void *dst, const void *src)
{
    asm volatile("cp.async.cg.shared.global [%0], [%1], 16;" ::"r"(smem_u32(dst)), "l"(src) : "memory");
}

// 4-byte asynchronous copy global -> shared (for sources without 16-byte alignment)
__device__ __forceinline__ void cp_async4(void *dst, const void *src)
{
    asm volatile("cp.async.ca.shared.global [%0], [%1], 4;" ::"r"(smem_u32(dst)), "l"(src) : "memory");
}

__device__ __forceinline__ void cp_async_commit() { asm volatile("cp.async.commit_group;" ::: "memory"); }
__device__ __forceinline__ void cp_async_wait_0() { asm volatile("cp.async.wait_group 0;" ::: "memory"); }
__device__ __forceinline__ void cp_async_wait_1() { asm volatile("cp.async.wait_group 1;" ::: "memory"); }
__device__ __forceinline__ void cp_async_wait_2() { asm volatile("cp.async.wait_group 2;" ::: "memory"); }
__device__ __forceinline__ void cp_async_wait_3() { asm volatile("cp.async.wait_group 3;" ::: "memory"); }

__device__ __forceinline__ void fence_proxy_async()
{
    asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
}

__device__ __forceinline__ unsigned ld_acquire_u32(const unsigned *p)
{
    unsigned v;
    asm volatile("ld.acquire.gpu.global.u32 %0, [%1];" : "=r"(v) : "l"(p) : "memory");
    return v;
}

__device__ __forceinline__ void st_release_u32(unsigned *p, unsigned v)
{
    asm volatile("st.release.gpu.global.u32 [%0], %1;" ::"l"(p), "r"(v) : "memory");
}

constexpr unsigned SPIN_LIMIT = 1u << 22;    // polls of >= 64 ns each: roughly a second at most

// dst = later o earlier for aggregates in shared memory, one warp; (A2,b2)o(A1,b1) = (A2 A1, A2 b1 + b2)
template <int N>
__device__ __forceinline__ void combine_smem(float *dst, const float *later, const float *earlier, int lane)
{
    constexpr int AGG = N * N + N;
    for (int o = lane; o < AGG; o += 32) {
        float acc;
        if (o < N * N) {
            const int i = o / N, j = o % N;
            acc = 0.0f;
#pragma unroll
            for (int k = 0; k < N; ++k) acc = fmaf(later[i * N + k], earlier[k * N + j], acc);
        } else {
            const int i = o - N * N;
            acc = later[N * N + i];
#pragma unroll
            for (int k = 0; k < N; ++k) acc = fmaf(later[i * N + k], earlier[N * N + k], acc);
        }
        dst[o] = acc;
    }
    __syncwarp();
}

// out = A in + beta for an aggregate in shared memory; lanes < N each produce one row
template <int N>
__device__ __forceinline__ void matvec_smem(float *out, const float *agg, const float *in, int lane)
{
    float acc = 0.0f;
    if (lane < N) {
        acc = agg[N * N + lane];
#pragma unroll
        for (int k = 0; k < N; ++k) acc = fmaf(agg[lane * N + k], in[k], acc);
    }
    __syncwarp();            // out may alias in
    if (lane < N) out[lane] = acc;
    __syncwarp();
}

__device__ __forceinline__ unsigned long long ld_relaxed_u64(const unsigned long long *p)
{
    unsigned long long v;
    asm volatile("ld.relaxed.gpu.global.u64 %0, [%1];" : "=l"(v) : "l"(p) : "memory");
    return v;
}

__device__ __forceinline__ void st_relaxed_u64(unsigned long long *p, unsigned long long v)
{
    asm volatile("st.relaxed.gpu.global.u64 [%0], %1;" ::"l"(p), "l"(v) : "memory");
}

// Geometry of one tile in shared memory.
//   run-padded (n >= 4): run r (= chain r) holds the run's positions in ascending t; scan step q
//                        of the run sits at local index q (forward) or cnt-1-q (reverse).
//   dense (n <= 2):      forward: position s0+u at slot u; reverse: ascending t, right-aligned in
//                        the buffer, so scan offset p = chain*S+q sits at slot L-1-p (keeps the
//                        128-bit groups of the n = 1 path aligned).
template <int N, bool REV> struct TileGeom {
    using C = OnePass<N>;
    int s0, Lt, T;
    __device__ __forceinline__ int run_cnt(int r) const { return min(C::S, max(0, Lt - r * C::S)); }
    __device__ __forceinline__ int dense_slot(int p) const { return REV ? (C::L - 1 - p) : p; }
    __device__ __forceinline__ int low_slot() const { return (REV && !C::PADDED) ? (C::L - Lt) : 0; }
    __device__ __forceinline__ int b_off(int chain, int q, int cnt) const
    {
        if constexpr (C::PADDED) return chain * C::BRUN + (REV ? cnt - 1 - q : q) * N;
        else return dense_slot(chain * C::S + q) * N;
    }
    __device__ __forceinline__ int j_off(int chain, int q, int cnt) const
    {
        if constexpr (C::PADDED) return chain * C::JRUN + (REV ? cnt - 1 - q : q) * N * N;
        else return dense_slot(chain * C::S + q) * N * N;
    }
    // run and local index of ascending-t index u of the tile (run-padded layout)
    __device__ __forceinline__ void locate(int u, int &r, int &li) const
    {
        if (!REV) { r = u / C::S; li = u - r * C::S; }
        else { const int ps = Lt - 1 - u; r = ps / C::S; li = run_cnt(r) - 1 - (ps - r * C::S); }
    }
    // float offset into sB of component i at ascending-t index u
    __device__ __forceinline__ int out_off(int u, int i) const
    {
        if constexpr (C::PADDED) { int r, li; locate(u, r, li); return r * C::BRUN + li * N + i; }
        else return (low_slot() + u) * N + i;
    }
    // float offset into sJ of the matrix at ascending index u of the tile's J range
    __device__ __forceinline__ int jmat_off(int u) const
    {
        if constexpr (C::PADDED) { int r, li; locate(u, r, li); return r * C::JRUN + li * N * N; }
        else return (low_slot() + u) * N * N;
    }
    __device__ __forceinline__ size_t t_lo() const { return REV ? (size_t)(T - s0 - Lt) : (size_t)s0; }
};

// one step of a chain from the staged tile: M = J (forward) or J^T (reverse; identity at scan position 0)
template <int N, bool REV>
__device__ __forceinline__ void load_chain_step(const float *sJ, const float *sB, const TileGeom<N, REV> &tg, int chain,
                                                int q, int cnt, float (&M)[N][N], float (&bq)[N])
{
    const float *Je = sJ + tg.j_off(chain, q, cnt);
    const float *bv = sB + tg.b_off(chain, q, cnt);
    const bool ident = REV && (tg.s0 + chain * OnePass<N>::S + q == 0);
    if constexpr (N == 2) {
        const float4 f = *reinterpret_cast<const float4 *>(Je);
        const float2 g = *reinterpret_cast<const float2 *>(bv);
        M[0][0] = f.x; M[0][1] = REV ? f.z : f.y; M[1][0] = REV ? f.y : f.z; M[1][1] = f.w;
        bq[0] = g.x; bq[1] = g.y;
    } else {
        static_assert(N == 2 || N == 4, "chain steps are read as 128-bit words");
        float R[4][4];
#pragma unroll
        for (int i = 0; i < 4; ++i) {
            const float4 f = reinterpret_cast<const float4 *>(Je)[i];
            R[i][0] = f.x; R[i][1] = f.y; R[i][2] = f.z; R[i][3] = f.w;
        }
#pragma unroll
        for (int i = 0; i < 4; ++i)
#pragma unroll
            for (int k = 0; k < 4; ++k) M[i][k] = REV ? R[k][i] : R[i][k];
        const float4 g = *reinterpret_cast<const float4 *>(bv);
        bq[0] = g.x; bq[1] = g.y; bq[2] = g.z; bq[3] = g.w;
    }
    if (ident) {
#pragma unroll
        for (int i = 0; i < N; ++i)
#pragma unroll
            for (int k = 0; k < N; ++k) M[i][k] = (i == k) ? 1.0f : 0.0f;
    }
}

// ---- n <= 4: one thread per chain; aggregates live in registers and are combined by warp shuffles
template <int N> struct RegAgg { float A[N][N]; float be[N]; };

template <int N> __device__ __forceinline__ void ragg_identity(RegAgg<N> &r)
{
#pragma unroll
    for (int i = 0; i < N; ++i) {
        r.be[i] = 0.0f;
#pragma unroll
        for (int j = 0; j < N; ++j) r.A[i][j] = (i == j) ? 1.0f : 0.0f;
    }
}

// r <- later o r
template <int N> __device__ __forceinline__ void ragg_push(RegAgg<N> &r, const float (&M)[N][N], const float (&b)[N])
{
    RegAgg<N> o;
#pragma unroll
    for (int i = 0; i < N; ++i) {
        o.be[i] = b[i];
#pragma unroll
        for (int k = 0; k < N; ++k) o.be[i] = fmaf(M[i][k], r.be[k], o.be[i]);
#pragma unroll
        for (int j = 0; j < N; ++j) {
            float acc = 0.0f;
#pragma unroll
            for (int k = 0; k < N; ++k) acc = fmaf(M[i][k], r.A[k][j], acc);
            o.A[i][j] = acc;
        }
    }
    r = o;
}

template <int N> __device__ __forceinline__ RegAgg<N> ragg_shfl_up(const RegAgg<N> &r, int d)
{
    RegAgg<N> o;
#pragma unroll
    for (int i = 0; i < N; ++i) {
        o.be[i] = __shfl_up_sync(0xffffffffu, r.be[i], d);
#pragma unroll
        for (int j = 0; j < N; ++j) o.A[i][j] = __shfl_up_sync(0xffffffffu, r.A[i][j], d);
    }
    return o;
}

// inclusive scan over the first W lanes of a warp (lane l ends with agg_l o ... o agg_0; the other
// lanes hold identities); returns the exclusive prefix (identity in lane 0) in `excl`
template <int N, int W = 32>
__device__ __forceinline__ void ragg_warp_scan(RegAgg<N> &r, RegAgg<N> &excl, int lane)
{
#pragma unroll
    for (int d = 1; d < W; d <<= 1) {
        RegAgg<N> p = ragg_shfl_up<N>(r, d);
        if (lane >= d) {
            RegAgg<N> e = p;            // earlier part
            ragg_push<N>(e, r.A, r.be);  // e <- r o e
            r = e;
        }
    }
    excl = ragg_shfl_up<N>(r, 1);
    if (lane == 0) ragg_identity<N>(excl);
}

template <int N> __device__ __forceinline__ void ragg_store(float *dst, const RegAgg<N> &r)
{
#pragma unroll
    for (int i = 0; i < N; ++i) {
        dst[N * N + i] = r.be[i];
#pragma unroll
        for (int j = 0; j < N; ++j) dst[i * N + j] = r.A[i][j];
    }
}

template <int N> __device__ __forceinline__ void ragg_load(RegAgg<N> &r, const float *src)
{
#pragma unroll
    for (int i = 0; i < N; ++i) {
        r.be[i] = src[N * N + i];
#pragma unroll
        for (int j = 0; j < N; ++j) r.A[i][j] = src[i * N + j];
    }
}

// y <- A y + beta
template <int N> __device__ __forceinline__ void ragg_apply(const RegAgg<N> &r, float (&y)[N])
{
    float o[N];
#pragma unroll
    for (int i = 0; i < N; ++i) {
        o[i] = r.be[i];
#pragma unroll
        for (int k = 0; k < N; ++k) o[i] = fmaf(r.A[i][k], y[k], o[i]);
    }
#pragma unroll
    for (int i = 0; i < N; ++i) y[i] = o[i];
}

// Flag polling shared by workers and resolvers: true while the run should go on.
// The limit is SPIN_LIMIT unless the launch carries its own (a.spin_limit: used by the test that makes
// a wait run out).
__device__ __forceinline__ bool keep_spinning(const ScanArgs &a, unsigned &spins)
{
    __nanosleep(64);
    const unsigned limit = a.spin_limit ? a.spin_limit : SPIN_LIMIT;
    if (++spins > limit) { atomicOr(&a.st->flags, FLAG_TIMEOUT); return false; }
    if ((spins & 255u) == 0 && (*(volatile unsigned *)&a.st->flags & FLAG_TIMEOUT)) return false;
    return true;
}

constexpr unsigned long long LL_FLAG = 1ull << 32;     // "entering state present" marker

// Resolver role with aggregates published as 64-bit {value, flag} words: warp `rw` of `nrw` serves
// sequences rw, rw + nrw, ...  A visit loads the words of the next WIN tiles of a sequence in one
// round trip, takes the leading tiles whose words are all present, clears those words for the next
// launch, and walks them, Y <- A Y + beta, writing the state entering every tile (lane i holds Y[i]).
template <int N>
__device__ void resolver_ll_loop(const ScanArgs &a, const OnePassWs &w, float *stage_all, int rw, int nrw, int lane)
{
    if (a.no_resolve) return;     // (wait-expiry test: nobody publishes entering states)
    using C = OnePass<N>;
    constexpr int AGG = C::AGG, NN = N * N;
    constexpr int WIN = 16;                         // tiles looked at per visit
    constexpr int PER = WIN * AGG / 32;             // words per lane
    static_assert((WIN * AGG) % 32 == 0 && WIN < 32, "window of whole words per lane");
    float *stage = stage_all + (threadIdx.x >> 5) * 32 * AGG;
    int nseq = 0;
    int pos[C::MAX_SEQ_PER_WARP];
    float yv[C::MAX_SEQ_PER_WARP];              // lane i < N: component i of the sequence's running state
#pragma unroll
    for (int k = 0; k < C::MAX_SEQ_PER_WARP; ++k) {
        pos[k] = 0; yv[k] = 0.0f;
        const int s = rw + k * nrw;
        if (s < a.B) {
            nseq = k + 1;
            if (lane < N && a.y0) yv[k] = a.y0[(size_t)s * N + lane];
        }
    }
    int remaining = nseq;
    unsigned spins = 0;
    while (remaining > 0) {
        bool progressed = false;
#pragma unroll
        for (int k = 0; k < C::MAX_SEQ_PER_WARP; ++k) {
            if (k >= nseq) break;
            const int c0 = pos[k];
            if (c0 >= w.nch) continue;
            const int s = rw + k * nrw;
            unsigned long long *words = reinterpret_cast<unsigned long long *>(w.aggs) + ((size_t)s * w.nch + c0) * AGG;
            const int nt = min(WIN, w.nch - c0);
            const int total = nt * AGG;
            unsigned long long v[PER];
#pragma unroll
            for (int u = 0; u < PER; ++u) {
                const int i = lane + 32 * u;
                v[u] = (i < total) ? ld_relaxed_u64(words + i) : 0ull;
            }
            unsigned missing = ~0u << nt;           // tiles beyond the window or the sequence
#pragma unroll
            for (int u = 0; u < PER; ++u) {
                const int i = lane + 32 * u;
                if (i < total && (v[u] >> 32) == 0ull) missing |= 1u << (i / AGG);
            }
            missing = __reduce_or_sync(0xffffffffu, missing);
            const int cnt = __ffs(missing) - 1;     // leading tiles with every word present
            if (cnt == 0) continue;
            progressed = true;
#pragma unroll
            for (int u = 0; u < PER; ++u) {
                const int i = lane + 32 * u;
                if (i < cnt * AGG) {
                    stage[i] = __uint_as_float((unsigned)(v[u] & 0xffffffffull));
                    st_relaxed_u64(words + i, 0ull);                 // consumed: cleared for the next launch
                }
            }
            __syncwarp();
            unsigned long long *out = w.starts + ((size_t)s * w.nch + c0) * N;
            float y = yv[k];
            for (int q = 0; q < cnt; ++q) {
                if (lane < N) st_relaxed_u64(out + q * N + lane, LL_FLAG | (unsigned long long)__float_as_uint(y));
                const float *ag = stage + q * AGG;
                float acc = (lane < N) ? ag[NN + lane] : 0.0f;
#pragma unroll
                for (int i = 0; i < N; ++i) {
                    const float yi = __shfl_sync(0xffffffffu, y, i);
                    if (lane < N) acc = fmaf(ag[lane * N + i], yi, acc);
                }
                y = acc;
            }
            yv[k] = y;
            __syncwarp();
            pos[k] = c0 + cnt;
            if (pos[k] >= w.nch) --remaining;
        }
        if (progressed) spins = 0;
        else if (!keep_spinning(a, spins)) return;
    }
}

template <int N, bool REV>
__global__ void __launch_bounds__(OnePass<N>::THREADS, 3) scan_onepass_kernel(ScanArgs a, OnePassWs w)
{
    using C = OnePass<N>;
    constexpr int S = C::S, CHAINS = C::CHAINS;
    constexpr int AGG = C::AGG, WARPS = C::WARPS, NN = N * N;
    constexpr int Q = C::Q, PEND = C::PEND;
    static_assert(N <= 2, "thread-per-chain kernel with a queue of pending tiles: n = 4 and above have their own kernels");

    extern __shared__ __align__(16) float smem_raw[];
    float *sJ = (float *)(((uintptr_t)smem_raw + 127) & ~(uintptr_t)127);
    float *sB = sJ + C::JBUF;
    float *pend = sB + C::BBUF;                // Q x { chain prefixes, warp prefixes }
    float *tmp = pend + Q * PEND;
    float *ystart = tmp + WARPS * 2 * AGG;
    uint64_t *bar = (uint64_t *)(((uintptr_t)(ystart + N) + 15) & ~(uintptr_t)15);
    __shared__ int s_kind, s_seq, s_c, s_slot, s_abort, s_role, s_done;

    pdl_prologue();
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const int chain = tid;
    const int T = a.T;

    // the role ticket and the loop-ended word travel together (one round trip; a ticket taken by a
    // launch that then returns is harmless: the counters are rewound before the next evaluation)
    if (tid == 0) {
        const unsigned ticket = atomicAdd(&a.st->role_counter, 1u);
        s_done = loop_ended(a.st) ? 1 : 0;
        mbar_init(bar, 1);
        s_abort = 0;
        s_role = (int)ticket;
    }
    fence_proxy_async();
    __syncthreads();
    if (s_done) return;
    if (s_role < w.resolvers) {
        resolver_ll_loop<N>(a, w, sJ, s_role * WARPS + warp, w.resolvers * WARPS, lane);
        __syncthreads();
        if (tid == 0) scan_epilogue(a.st);
        return;
    }
    unsigned phase = 0;
    unsigned mb = 0;          // running max |y - yold| bits of this thread

    // id -> (seq, chunk); chunk < 0 when the id is padding of the last window
    auto decode = [&](unsigned id, int &seq, int &c) {
        const unsigned j = id % (unsigned)w.Wd;
        const unsigned ws_ = id / (unsigned)w.Wd;
        seq = (int)(ws_ % (unsigned)a.B);
        const unsigned win = ws_ / (unsigned)a.B;
        c = (int)(win * (unsigned)w.Wd + j);
        if (c >= w.nch) c = -1;
    };

    // pending queue (thread 0 only): tiles whose A item has run
    int q_seq[Q], q_c[Q], q_head = 0, q_cnt = 0;
    bool exhausted = false;
    // tile ids come from the same counter as the role tickets (ticket - resolvers): a worker's ticket
    // is its first tile id (no second atomic before the first tile), and ids are still handed out in
    // order to running CTAs only
    bool first_claim = true;

    for (;;) {
        __syncthreads();      // previous item done with shared memory and with the s_* words
        if (tid == 0) {
            // next item: the oldest pending tile's B item as soon as its entering state is
            // there (or when the queue is full / no tiles are left), otherwise a new tile's A item
            int kind = -1, seq = -1, c = -1, slot = 0;
            bool want_b = false;
            if (q_cnt > 0) {
                want_b = (q_cnt == Q) || exhausted;
                if (!want_b)
                    want_b = ld_relaxed_u64(w.starts + ((size_t)q_seq[q_head] * w.nch + q_c[q_head]) * N) != 0ull;
            }
            if (!want_b && !exhausted) {
                for (;;) {
                    unsigned id;
                    if (first_claim) { id = (unsigned)(s_role - w.resolvers); first_claim = false; }
                    else id = atomicAdd(&a.st->role_counter, 1u) - (unsigned)w.resolvers;
                    if (id >= w.total_ids) { c = -1; break; }
                    decode(id, seq, c);
                    if (c >= 0) break;
                }
                if (c >= 0) {
                    kind = 0;
                    slot = (q_head + q_cnt) % Q;
                    q_seq[slot] = seq; q_c[slot] = c; ++q_cnt;
                } else {
                    exhausted = true;
                    want_b = q_cnt > 0;
                }
            }
            if (want_b) {
                kind = 1; slot = q_head; seq = q_seq[q_head]; c = q_c[q_head];
                q_head = (q_head + 1) % Q; --q_cnt;
            }
            s_kind = kind; s_seq = seq; s_c = c; s_slot = slot;
        }
        __syncthreads();
        if (s_kind < 0 || s_abort) break;
        const int kind = s_kind, seq = s_seq, c = s_c;
        float *agg = pend + s_slot * PEND;          // exclusive chain prefixes within the warp
        float *wagg = agg + CHAINS * AGG;           // exclusive warp prefixes
        TileGeom<N, REV> tg;
        tg.s0 = c * C::L;
        tg.Lt = min(C::L, T - tg.s0);
        tg.T = T;
        const int s0 = tg.s0, Lt = tg.Lt;
        const size_t p_lo = tg.t_lo();                                  // first b element of the tile
        const size_t j_lo = REV ? p_lo + 1 : p_lo;                      // first J element of the tile
        const int jcnt_tile = (REV && s0 == 0) ? Lt - 1 : Lt;           // (reverse: J[T] does not exist)
        const size_t tile_index = (size_t)seq * w.nch + c;
        const float *Jt_src = a.J + ((size_t)seq * T + j_lo) * NN;
        const float *bt_src = a.b + ((size_t)seq * T + p_lo) * N;
        // ------------------------------------------------ stage the tile (bulk copies where aligned)
        {
            const unsigned jb = (unsigned)jcnt_tile * NN * 4u, bb = (unsigned)Lt * N * 4u;
            float *jd = sJ + tg.low_slot() * NN, *bd = sB + tg.low_slot() * N;
            const bool jbulk = jb && ((uintptr_t)Jt_src & 15) == 0 && (jb & 15) == 0 && ((uintptr_t)jd & 15) == 0;
            const bool bbulk = ((uintptr_t)bt_src & 15) == 0 && (bb & 15) == 0 && ((uintptr_t)bd & 15) == 0;
            if (tid == 0) {
                fence_proxy_async();
                mbar_arrive_expect_tx(bar, (jbulk ? jb : 0u) + (bbulk ? bb : 0u));
                if (jbulk) bulk_g2s(jd, Jt_src, jb, bar);
                if (bbulk) bulk_g2s(bd, bt_src, bb, bar);
            }
            // sources that are not 16-byte aligned (the reverse scan of n = 1 reads J one element on): 4-byte
            // asynchronous copies, one instruction per element and no registers in between
            if (!jbulk) for (int i = tid; i < jcnt_tile * NN; i += C::THREADS) cp_async4(jd + i, Jt_src + i);
            if (!bbulk) for (int i = tid; i < Lt * N; i += C::THREADS) cp_async4(bd + i, bt_src + i);
            cp_async_commit();
        }
        // B item: while the copies fly, warp 1 fetches the state entering the tile ({value, flag} words)
        if (kind == 1 && warp == 1) {
            const unsigned long long *src = w.starts + tile_index * N;
            unsigned spins = 0;
            bool ok = true;
            for (;;) {
                const unsigned long long v = (lane < N) ? ld_relaxed_u64(src + lane) : LL_FLAG;
                if (__all_sync(0xffffffffu, v != 0ull)) {
                    if (lane < N) {
                        ystart[lane] = __uint_as_float((unsigned)(v & 0xffffffffull));
                        st_relaxed_u64(w.starts + tile_index * N + lane, 0ull);     // consumed: cleared for the next launch
                    }
                    break;
                }
                if (!keep_spinning(a, spins)) { ok = false; break; }
            }
            if (!__all_sync(0xffffffffu, ok)) s_abort = 1;
        }
        cp_async_wait_0();      // this thread's 4-byte copies, if any
        {
            unsigned spins = 0;
            while (!mbar_try_wait(bar, phase)) {
                if (++spins > (SPIN_LIMIT >> 2)) { atomicOr(&a.st->flags, FLAG_TIMEOUT); s_abort = 1; break; }
            }
            phase ^= 1u;
        }
        __syncthreads();      // plain-copied data, ystart and s_abort visible
        if (s_abort) break;

        const int cnt = tg.run_cnt(chain);
        {
            // ============================================ one thread per chain
            if (kind == 0) {
                RegAgg<N> r;
                ragg_identity<N>(r);
                if constexpr (N == 1) {
#pragma unroll
                    for (int q4 = 0; q4 < S / 4; ++q4) {
                        const int p = chain * S + 4 * q4;
                        const int base = REV ? (C::L - 4 - p) : p;
                        const float4 j4 = *reinterpret_cast<const float4 *>(sJ + base);
                        const float4 b4 = *reinterpret_cast<const float4 *>(sB + base);
                        const float jj[4] = {REV ? j4.w : j4.x, REV ? j4.z : j4.y, REV ? j4.y : j4.z, REV ? j4.x : j4.w};
                        const float bb[4] = {REV ? b4.w : b4.x, REV ? b4.z : b4.y, REV ? b4.y : b4.z, REV ? b4.x : b4.w};
#pragma unroll
                        for (int k = 0; k < 4; ++k) {
                            if (4 * q4 + k < cnt) {
                                const float jv = (REV && s0 + p + k == 0) ? 1.0f : jj[k];
                                r.A[0][0] = jv * r.A[0][0];
                                r.be[0] = fmaf(jv, r.be[0], bb[k]);
                            }
                        }
                    }
                } else {
#pragma unroll
                    for (int q = 0; q < S; ++q) {
                        if (q < cnt) {
                            float M[N][N], bq[N];
                            load_chain_step<N, REV>(sJ, sB, tg, chain, q, cnt, M, bq);
                            ragg_push<N>(r, M, bq);
                        }
                    }
                }
                RegAgg<N> ex;
                ragg_warp_scan<N>(r, ex, lane);
                ragg_store<N>(agg + chain * AGG, ex);              // exclusive prefix inside the warp
                if (lane == 31) ragg_store<N>(tmp + warp * AGG, r);   // warp aggregate
                __syncthreads();
                if (warp == 0) {
                    RegAgg<N> wr;
                    if (lane < WARPS) ragg_load<N>(wr, tmp + lane * AGG);
                    else ragg_identity<N>(wr);
                    RegAgg<N> wex;
                    ragg_warp_scan<N, WARPS>(wr, wex, lane);
                    if (lane < WARPS) ragg_store<N>(wagg + lane * AGG, wex);   // exclusive prefix over warps
                    if (lane == WARPS - 1) {
                        // tile aggregate as {value, flag} words: no fence, one round trip for the reader
                        unsigned long long *dst = reinterpret_cast<unsigned long long *>(w.aggs) + tile_index * AGG;
#pragma unroll
                        for (int i = 0; i < N; ++i) {
#pragma unroll
                            for (int j = 0; j < N; ++j)
                                st_relaxed_u64(dst + i * N + j, LL_FLAG | (unsigned long long)__float_as_uint(wr.A[i][j]));
                            st_relaxed_u64(dst + N * N + i, LL_FLAG | (unsigned long long)__float_as_uint(wr.be[i]));
                        }
                    }
                }
                continue;
            }
            {
                float y[N];
#pragma unroll
                for (int k = 0; k < N; ++k) y[k] = ystart[k];
                RegAgg<N> e;
                ragg_load<N>(e, wagg + warp * AGG);
                ragg_apply<N>(e, y);
                ragg_load<N>(e, agg + chain * AGG);
                ragg_apply<N>(e, y);
                if constexpr (N == 1) {
                    float yv = y[0];
#pragma unroll
                    for (int q4 = 0; q4 < S / 4; ++q4) {
                        const int p = chain * S + 4 * q4;
                        const int base = REV ? (C::L - 4 - p) : p;
                        const float4 j4 = *reinterpret_cast<const float4 *>(sJ + base);
                        float4 b4 = *reinterpret_cast<const float4 *>(sB + base);
                        const float jj[4] = {REV ? j4.w : j4.x, REV ? j4.z : j4.y, REV ? j4.y : j4.z, REV ? j4.x : j4.w};
                        float bb[4] = {REV ? b4.w : b4.x, REV ? b4.z : b4.y, REV ? b4.y : b4.z, REV ? b4.x : b4.w};
#pragma unroll
                        for (int k = 0; k < 4; ++k) {
                            if (4 * q4 + k < cnt) {
                                const float jv = (REV && s0 + p + k == 0) ? 1.0f : jj[k];
                                yv = fmaf(jv, yv, bb[k]);
                                bb[k] = yv;
                            }
                        }
                        if (REV) { b4.w = bb[0]; b4.z = bb[1]; b4.y = bb[2]; b4.x = bb[3]; }
                        else { b4.x = bb[0]; b4.y = bb[1]; b4.z = bb[2]; b4.w = bb[3]; }
                        if (4 * q4 < cnt) *reinterpret_cast<float4 *>(sB + base) = b4;
                    }
                } else {
#pragma unroll
                    for (int q = 0; q < S; ++q) {
                        if (q < cnt) {
                            float M[N][N], bq[N];
                            load_chain_step<N, REV>(sJ, sB, tg, chain, q, cnt, M, bq);
                            float yn[N];
#pragma unroll
                            for (int i = 0; i < N; ++i) {
                                yn[i] = bq[i];
#pragma unroll
                                for (int k = 0; k < N; ++k) yn[i] = fmaf(M[i][k], y[k], yn[i]);
                            }
#pragma unroll
                            for (int i = 0; i < N; ++i) y[i] = yn[i];
                            float *bv = sB + tg.b_off(chain, q, cnt);
                            if constexpr (N == 2) *reinterpret_cast<float2 *>(bv) = make_float2(yn[0], yn[1]);
                            else *reinterpret_cast<float4 *>(bv) = make_float4(yn[0], yn[1], yn[2], yn[3]);
                        }
                    }
                }
            }
            __syncthreads();
        }

        // ------------------------------------------------ stream y out (+ max |y - yold|)
        {
            const size_t gbase = ((size_t)seq * T + tg.t_lo()) * N;
            float *yo = a.y + gbase;
            const float *yold = a.yold ? a.yold + gbase : nullptr;
            const int total = Lt * N;
            const bool vec = (N >= 4 || (tg.low_slot() * N) % 4 == 0) && (((uintptr_t)yo & 15) == 0) &&
                             ((total & 3) == 0) && (!yold || ((uintptr_t)yold & 15) == 0);
            if (vec) {
                for (int g4 = tid; g4 < total / 4; g4 += C::THREADS) {
                    const int g = 4 * g4;
                    const float4 val = *reinterpret_cast<const float4 *>(sB + tg.out_off(g / N, g % N));
                    if (yold) {
                        const float4 o = __ldg(reinterpret_cast<const float4 *>(yold) + g4);
                        mb = max(mb, absdiff_bits(val.x, o.x)); mb = max(mb, absdiff_bits(val.y, o.y));
                        mb = max(mb, absdiff_bits(val.z, o.z)); mb = max(mb, absdiff_bits(val.w, o.w));
                    }
                    reinterpret_cast<float4 *>(yo)[g4] = val;
                }
            } else {
                for (int g = tid; g < total; g += C::THREADS) {
                    const float val = sB[tg.out_off(g / N, g % N)];
                    if (yold) mb = max(mb, absdiff_bits(val, yold[g]));
                    yo[g] = val;
                }
            }
        }
    }
    if (a.yold) {
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) mb = max(mb, __shfl_xor_sync(0xffffffffu, mb, o));
        if (lane == 0 && mb) { atomicMax(&a.st->err_bits, mb); __threadfence(); }
    }
    __syncthreads();
    if (tid == 0) scan_epilogue(a.st);
}

}  // namespace deer
