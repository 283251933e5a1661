// Single-pass chunked scan of the linear recurrence for n in {1, 2, 4, 8}:
// J and b are read from HBM once, y written once.
//
//   * One persistent kernel.  Every tile of L consecutive positions of one
//     sequence is visited twice by a worker CTA: an A item (stage the tile,
//     fold it into the tile aggregate, publish the aggregate) and, a few items
//     later, a B item (stage the tile again -- by then from L2 --, replay it
//     from its entering state, write y).  A items never wait on anything; the
//     entering states are produced by resolver warps (a few CTAs that took the
//     first role tickets) which walk each sequence's published aggregates in
//     order.  Workers therefore hold no data while a dependency is in flight.
//   * Tiles are staged in shared memory by bulk asynchronous copies
//     (cp.async.bulk + mbarrier).  The data of the tile that will be taken one
//     grid-round later is prefetched into L2 (cp.async.bulk.prefetch.L2), so
//     HBM stays busy while the SMs compute.
//   * A chain is LPC lanes that own S consecutive positions.  Each lane keeps
//     COLS = n / LPC columns of the running product A (and the whole vector
//     beta, redundantly) in registers and multiplies the next J_t, broadcast
//     from shared memory, onto them:  (A, beta) <- (J_t A, J_t beta + b_t).
//   * Bank conflicts: for n >= 4 every chain run is copied on its own and
//     padded by 16 bytes, which makes the run stride odd in 16-byte units; for
//     n <= 2 the tile is dense and S is chosen odd (n = 2) or S/4 odd (n = 1,
//     processed four positions per 128-bit load).
//   * Chain aggregates are combined per warp and per tile in shared memory
//     and kept there (a small queue of pending tiles) for the B item.
//   * Roles and tile ids are handed out by atomic counters to running CTAs
//     only, and a tile's B item depends only on A items of lower ids, which
//     their owners execute immediately after claiming: no co-residency
//     assumption is needed for progress.  Every wait is bounded all the same:
//     on expiry the kernel raises FLAG_TIMEOUT and all CTAs drain.
//   * In the B item the tile is replayed from its entering state (matrix-
//     vector work only), y overwrites b in shared memory and is streamed out
//     with coalesced stores fused with the max |y - y_old| reduction.
//
// Reverse scans (the adjoint) use the same kernel with reversed indexing and
// transposed register access.
#pragma once
#include "common.cuh"

namespace deer {

template <int N> struct OnePass {
    static constexpr int LPC = (N >= 4) ? 4 : N;       // lanes per chain
    static constexpr int COLS = N / LPC;               // columns of A per lane
    static constexpr int S = (N == 8) ? 5 : (N == 4) ? 24 : (N == 2) ? 39 : 60;   // positions per chain
    static constexpr int PAD = (N >= 4) ? 4 : 0;       // floats of padding after each chain run
    static constexpr int THREADS = 128;
    static constexpr int WARPS = THREADS / 32;
    static constexpr int CHAINS = THREADS / LPC;
    static constexpr int CPW = CHAINS / WARPS;         // chains per warp
    static constexpr int L = CHAINS * S;               // positions per tile
    static constexpr int JRUN = S * N * N + PAD;       // floats per chain run of J
    static constexpr int BRUN = S * N + PAD;           // floats per chain run of b / y
    static constexpr int AGG = N * N + N;              // floats of one aggregate (A row-major, then beta)
    static constexpr int Q = 2;                        // pending tiles (A done, B not yet) per CTA
    static constexpr int PEND = (CHAINS + WARPS) * AGG; // chain + warp aggregates kept per pending tile
    static constexpr int SM_FLOATS = CHAINS * JRUN + CHAINS * BRUN + Q * PEND + WARPS * 2 * AGG + AGG +
                                     CHAINS * N + WARPS * N + N + 4;
    static constexpr int MAX_SEQ_PER_WARP = 8;         // sequences one resolver warp can serve
    static_assert(32 * AGG <= (CHAINS * JRUN) / WARPS, "resolver staging must fit the tile buffer");
    static constexpr size_t SMEM = SM_FLOATS * sizeof(float) + 64;
    static_assert(N == 1 ? ((S / 4) % 2 == 1 && S % 4 == 0) : N == 2 ? (S % 2 == 1)
                  : ((JRUN / 4) % 2 == 1 && (BRUN / 4) % 2 == 1), "chain stride must avoid bank conflicts");
};

struct OnePassWs {
    unsigned *flags;     // [B*nch]   0 = nothing, 1 = aggregate published, 2 = entering state published
    float *aggs;         // [B*nch][n*n+n]
    float *starts;       // [B*nch][n]  state entering the tile
    int nch, Wd, nwin;   // tiles per sequence, tiles per sequence per window, windows
    unsigned total_ids;
    int resolvers;       // CTAs that take the resolver role
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

__device__ __forceinline__ void bulk_prefetch_l2(const void *src, unsigned bytes)
{
    asm volatile("cp.async.bulk.prefetch.L2.global [%0], %1;" ::"l"(src), "r"(bytes) : "memory");
}

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

// Geometry of one tile in the two shared-memory layouts.
//   padded (n >= 4): run r holds the run's positions in ascending t; scan step q of the
//                    run sits at local index q (forward) or cnt-1-q (reverse).
//   dense  (n <= 2): forward: position s0+u at slot u; reverse: ascending t, right-aligned
//                    in the buffer, so scan offset p = chain*S+q sits at slot L-1-p.
template <int N, bool REV> struct TileGeom {
    using C = OnePass<N>;
    int s0, Lt, T;
    __device__ __forceinline__ int run_cnt(int r) const { return min(C::S, max(0, Lt - r * C::S)); }
    // element slot (in elements) for the dense layout
    __device__ __forceinline__ int dense_slot(int p) const { return REV ? (C::L - 1 - p) : p; }
    __device__ __forceinline__ int dense_base() const { return REV ? (C::L - Lt) : 0; }   // slot of the lowest t
    // float offset into sB / sJ(elements * NN) for scan step q of chain `chain`
    __device__ __forceinline__ int b_off(int chain, int q, int cnt) const
    {
        if constexpr (C::PAD > 0) return chain * C::BRUN + (REV ? cnt - 1 - q : q) * N;
        else return dense_slot(chain * C::S + q) * N;
    }
    __device__ __forceinline__ int j_off(int chain, int q, int cnt) const
    {
        if constexpr (C::PAD > 0) return chain * C::JRUN + (REV ? cnt - 1 - q : q) * N * N;
        else return dense_slot(chain * C::S + q) * N * N;
    }
    // float offset into sB of component i at ascending-t index u of the tile
    __device__ __forceinline__ int out_off(int u, int i) const
    {
        if constexpr (C::PAD > 0) {
            if (!REV) { const int r = u / C::S; return r * C::BRUN + (u - r * C::S) * N + i; }
            const int ps = Lt - 1 - u, r = ps / C::S, q = ps % C::S;
            return r * C::BRUN + (run_cnt(r) - 1 - q) * N + i;
        } else {
            return (dense_base() + u) * N + i;
        }
    }
    __device__ __forceinline__ size_t t_lo() const { return REV ? (size_t)(T - s0 - Lt) : (size_t)s0; }
};

// Flag polling shared by workers and resolvers: true while the run should go on.
__device__ __forceinline__ bool keep_spinning(StatusBlock *st, unsigned &spins)
{
    __nanosleep(64);
    if (++spins > SPIN_LIMIT) { atomicOr(&st->flags, FLAG_TIMEOUT); return false; }
    if ((spins & 255u) == 0 && (*(volatile unsigned *)&st->flags & FLAG_TIMEOUT)) return false;
    return true;
}

// Resolver role: warp `rw` of `nrw` serves sequences rw, rw + nrw, ...  For each it walks the
// published tile aggregates in order, Y <- A Y + beta, writing the state entering every tile.
template <int N>
__device__ void resolver_loop(const ScanArgs &a, const OnePassWs &w, float *stage_all, float *ybuf_all,
                              int rw, int nrw, int lane)
{
    using C = OnePass<N>;
    constexpr int AGG = C::AGG;
    float *stage = stage_all + (threadIdx.x >> 5) * 32 * AGG;
    float *ybuf = ybuf_all + (threadIdx.x >> 5) * C::MAX_SEQ_PER_WARP * N;
    int nseq = 0;
    int pos[C::MAX_SEQ_PER_WARP];
#pragma unroll
    for (int k = 0; k < C::MAX_SEQ_PER_WARP; ++k) {
        pos[k] = 0;
        const int s = rw + k * nrw;
        if (s < a.B) {
            nseq = k + 1;
            if (lane < N) ybuf[k * N + lane] = a.y0 ? a.y0[(size_t)s * N + lane] : 0.0f;
        }
    }
    __syncwarp();
    int remaining = nseq;
    unsigned spins = 0;
    while (remaining > 0) {
        bool progressed = false;
#pragma unroll 1
        for (int k = 0; k < nseq; ++k) {
            const int c0 = pos[k];
            if (c0 >= w.nch) continue;
            const int s = rw + k * nrw;
            unsigned *flags = w.flags + (size_t)s * w.nch;
            const int j = c0 + lane;
            const unsigned f = (j < w.nch) ? ld_acquire_u32(flags + j) : 0u;
            const unsigned m = __ballot_sync(0xffffffffu, f >= 1u);
            const int cnt = (m == 0xffffffffu) ? 32 : (__ffs(~m) - 1);      // contiguous published aggregates
            if (cnt == 0) continue;
            progressed = true;
            const float *src = w.aggs + ((size_t)s * w.nch + c0) * AGG;
            for (int i = lane; i < cnt * AGG; i += 32) stage[i] = __ldcg(src + i);
            __syncwarp();
            float *y = ybuf + k * N;
            float *out = w.starts + ((size_t)s * w.nch + c0) * N;
            for (int q = 0; q < cnt; ++q) {
                if (lane < N) out[q * N + lane] = y[lane];
                matvec_smem<N>(y, stage + q * AGG, y, lane);
            }
            __threadfence();
            __syncwarp();
            if (lane < cnt) st_release_u32(flags + c0 + lane, 2u);
            pos[k] = c0 + cnt;
            if (pos[k] >= w.nch) --remaining;
        }
        if (progressed) spins = 0;
        else if (!keep_spinning(a.st, spins)) return;
    }
}

template <int N, bool REV>
__global__ void __launch_bounds__(OnePass<N>::THREADS) scan_onepass_kernel(ScanArgs a, OnePassWs w)
{
    using C = OnePass<N>;
    constexpr int LPC = C::LPC, COLS = C::COLS, S = C::S, CHAINS = C::CHAINS, CPW = C::CPW;
    constexpr int JRUN = C::JRUN, BRUN = C::BRUN, AGG = C::AGG, WARPS = C::WARPS, NN = N * N;
    constexpr int Q = C::Q, PEND = C::PEND;
    constexpr bool PADDED = C::PAD > 0;

    extern __shared__ __align__(16) float smem[];
    float *sJ = smem;
    float *sB = sJ + CHAINS * JRUN;
    float *pend = sB + CHAINS * BRUN;          // Q x { chain aggregates, warp aggregates }
    float *tmp = pend + Q * PEND;
    float *tagg = tmp + WARPS * 2 * AGG;
    float *cstart = tagg + AGG;
    float *wstart = cstart + CHAINS * N;
    float *ystart = wstart + WARPS * N;
    uint64_t *bar = (uint64_t *)(((uintptr_t)(ystart + N) + 15) & ~(uintptr_t)15);
    __shared__ int s_kind, s_seq, s_c, s_slot, s_abort, s_role;

    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const int chain = tid / LPC, sub = tid % LPC;
    const unsigned chain_mask = (LPC == 32) ? 0xffffffffu : (((1u << LPC) - 1u) << (lane & ~(LPC - 1)));
    const int chain_lane0 = lane & ~(LPC - 1);
    const int T = a.T;

    if (tid == 0) {
        mbar_init(bar, 1);
        s_abort = 0;
        s_role = (int)atomicAdd(&a.st->role_counter, 1u);
    }
    fence_proxy_async();
    __syncthreads();
    if (s_role < w.resolvers) {
        resolver_loop<N>(a, w, sJ, sB, s_role * WARPS + warp, w.resolvers * WARPS, lane);
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
    // global ranges of one tile: J elements [j_lo, j_lo + jcnt), b elements [p_lo, p_lo + Lt)
    auto tile_ranges = [&](int c, int &s0, int &Lt, size_t &p_lo, size_t &j_lo, int &jcnt) {
        s0 = c * C::L;
        Lt = min(C::L, T - s0);
        p_lo = REV ? (size_t)(T - s0 - Lt) : (size_t)s0;
        j_lo = REV ? p_lo + 1 : p_lo;
        jcnt = (REV && s0 == 0) ? Lt - 1 : Lt;
    };

    // pending queue (thread 0 only): tiles whose A item is done
    int q_seq[Q], q_c[Q], q_head = 0, q_cnt = 0;
    bool exhausted = false;

    for (;;) {
        __syncthreads();      // previous item done with shared memory and with the s_* words
        if (tid == 0) {
            int kind = -1, seq = -1, c = -1, slot = 0;
            bool want_b = false;
            if (q_cnt > 0) {
                want_b = (q_cnt == Q) || exhausted;
                if (!want_b)
                    want_b = ld_acquire_u32(w.flags + (size_t)q_seq[q_head] * w.nch + q_c[q_head]) == 2u;
            }
            if (!want_b && !exhausted) {
                unsigned id = 0;
                for (;;) {
                    id = atomicAdd(&a.st->tile_counter, 1u);
                    if (id >= w.total_ids) { c = -1; break; }
                    decode(id, seq, c);
                    if (c >= 0) break;
                }
                if (c >= 0) {
                    kind = 0;
                    slot = (q_head + q_cnt) % Q;
                    q_seq[slot] = seq; q_c[slot] = c; ++q_cnt;
                    // warm L2 with the tile that some CTA will take one grid-round from now
                    if (id + gridDim.x < w.total_ids) {
                        int pseq, pc;
                        decode(id + gridDim.x, pseq, pc);
                        if (pc >= 0) {
                            int ps0, pLt, pj; size_t pp, pjl;
                            tile_ranges(pc, ps0, pLt, pp, pjl, pj);
                            const float *jsrc = a.J + ((size_t)pseq * T + pjl) * NN;
                            const float *bsrc = a.b + ((size_t)pseq * T + pp) * N;
                            const unsigned jb = (unsigned)pj * NN * 4u, bb = (unsigned)pLt * N * 4u;
                            if (jb && ((uintptr_t)jsrc & 15) == 0 && (jb & 15) == 0) bulk_prefetch_l2(jsrc, jb);
                            if (((uintptr_t)bsrc & 15) == 0 && (bb & 15) == 0) bulk_prefetch_l2(bsrc, bb);
                        }
                    }
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
        float *agg = pend + s_slot * PEND;          // chain aggregates of this tile
        float *wagg = agg + CHAINS * AGG;           // warp aggregates of this tile
        TileGeom<N, REV> tg;
        size_t p_lo, j_lo;
        int jcnt_tile;
        tile_ranges(c, tg.s0, tg.Lt, p_lo, j_lo, jcnt_tile);
        tg.T = T;
        const int s0 = tg.s0, Lt = tg.Lt;
        const size_t tile_index = (size_t)seq * w.nch + c;
        const float *Jt_src = a.J + ((size_t)seq * T + j_lo) * NN;
        const float *bt_src = a.b + ((size_t)seq * T + p_lo) * N;

        // ------------------------------------------------ stage the tile
        if constexpr (PADDED) {
            if (warp == 0) {          // one bulk copy per chain run of J (always 16-byte aligned for n >= 4)
                fence_proxy_async();
                unsigned bytes = 0;
#pragma unroll 1
                for (int r = lane; r < CHAINS; r += 32) {
                    int cnt = tg.run_cnt(r);
                    if (REV && s0 + r * S == 0) cnt -= 1;
                    if (cnt > 0) bytes += (unsigned)cnt * NN * 4u;
                }
#pragma unroll
                for (int o = 16; o > 0; o >>= 1) bytes += __shfl_xor_sync(0xffffffffu, bytes, o);
                if (lane == 0) mbar_arrive_expect_tx(bar, bytes);
                __syncwarp();
#pragma unroll 1
                for (int r = lane; r < CHAINS; r += 32) {
                    const int cnt = tg.run_cnt(r);
                    if (cnt <= 0) continue;
                    // ascending-t index of the run's first J element inside the tile's J range
                    int first = REV ? (Lt - (r * S + cnt)) : r * S;
                    int jc = cnt;
                    if (REV && s0 + r * S == 0) jc -= 1;
                    if (jc > 0) bulk_g2s(sJ + r * JRUN, Jt_src + (size_t)first * NN, (unsigned)jc * NN * 4u, bar);
                }
            }
            // b: coalesced 128-bit loads by everybody into the padded runs
            for (int g4 = tid; g4 < Lt * N / 4; g4 += C::THREADS) {
                const int g = 4 * g4;
                const float4 v = __ldg(reinterpret_cast<const float4 *>(bt_src) + g4);
                *reinterpret_cast<float4 *>(sB + tg.out_off(g / N, g % N)) = v;
            }
        } else {
            const unsigned jb = (unsigned)jcnt_tile * NN * 4u, bb = (unsigned)Lt * N * 4u;
            float *jd = sJ + tg.dense_base() * NN, *bd = sB + tg.dense_base() * N;
            const bool jbulk = jb && ((uintptr_t)Jt_src & 15) == 0 && (jb & 15) == 0 && ((uintptr_t)jd & 15) == 0;
            const bool bbulk = ((uintptr_t)bt_src & 15) == 0 && (bb & 15) == 0 && ((uintptr_t)bd & 15) == 0;
            if (tid == 0) {
                fence_proxy_async();
                mbar_arrive_expect_tx(bar, (jbulk ? jb : 0u) + (bbulk ? bb : 0u));
                if (jbulk) bulk_g2s(jd, Jt_src, jb, bar);
                if (bbulk) bulk_g2s(bd, bt_src, bb, bar);
            }
            if (!jbulk) for (int i = tid; i < jcnt_tile * NN; i += C::THREADS) jd[i] = __ldg(Jt_src + i);
            if (!bbulk) for (int i = tid; i < Lt * N; i += C::THREADS) bd[i] = __ldg(bt_src + i);
        }
        // B item: while the copies fly, one thread waits for the state entering the tile
        if (kind == 1 && tid == 32) {
            const unsigned *fl = w.flags + tile_index;
            unsigned spins = 0;
            bool ok = true;
            while (ld_acquire_u32(fl) != 2u) {
                if (!keep_spinning(a.st, spins)) { ok = false; break; }
            }
            if (ok) {
                __threadfence();
#pragma unroll
                for (int k = 0; k < N; ++k) ystart[k] = __ldcg(w.starts + tile_index * N + k);
            } else {
                s_abort = 1;
            }
        }
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
        if (kind == 0) {
            // -------------------------------------------- A item: chain aggregate in registers
            float A[N][COLS], be[N];
#pragma unroll
            for (int i = 0; i < N; ++i) {
                be[i] = 0.0f;
#pragma unroll
                for (int cc = 0; cc < COLS; ++cc) A[i][cc] = (i == sub * COLS + cc) ? 1.0f : 0.0f;
            }
            if constexpr (N == 1) {
                // four positions per 128-bit load; dense layout, groups are 16-byte aligned
                float am = 1.0f, bm = 0.0f;
#pragma unroll 1
                for (int q4 = 0; q4 < S / 4; ++q4) {
                    if (4 * q4 >= cnt) break;
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
                            am = jv * am;
                            bm = fmaf(jv, bm, bb[k]);
                        }
                    }
                }
                A[0][0] = am; be[0] = bm;
            } else {
#pragma unroll 1
                for (int q = 0; q < cnt; ++q) {
                    const bool ident = REV && (s0 + chain * S + q == 0);
                    const float *Je = sJ + tg.j_off(chain, q, cnt);
                    const float *bv = sB + tg.b_off(chain, q, cnt);
                    float bq[N];
                    if constexpr (N >= 4) {
#pragma unroll
                        for (int v = 0; v < N / 4; ++v) {
                            const float4 f = reinterpret_cast<const float4 *>(bv)[v];
                            bq[4 * v] = f.x; bq[4 * v + 1] = f.y; bq[4 * v + 2] = f.z; bq[4 * v + 3] = f.w;
                        }
                    } else {
                        const float2 f = *reinterpret_cast<const float2 *>(bv);
                        bq[0] = f.x; bq[1] = f.y;
                    }
                    if (q == 0) {
                        if (!ident) {
#pragma unroll
                            for (int i = 0; i < N; ++i)
#pragma unroll
                                for (int cc = 0; cc < COLS; ++cc) {
                                    const int j = sub * COLS + cc;
                                    A[i][cc] = REV ? Je[j * N + i] : Je[i * N + j];
                                }
                        }
#pragma unroll
                        for (int i = 0; i < N; ++i) be[i] = bq[i];
                        continue;
                    }
                    float Jr[NN];
#pragma unroll
                    for (int v = 0; v < NN / 4; ++v) {
                        const float4 f = reinterpret_cast<const float4 *>(Je)[v];
                        Jr[4 * v] = f.x; Jr[4 * v + 1] = f.y; Jr[4 * v + 2] = f.z; Jr[4 * v + 3] = f.w;
                    }
                    float An[N][COLS], bn[N];
#pragma unroll
                    for (int i = 0; i < N; ++i) {
                        bn[i] = bq[i];
#pragma unroll
                        for (int cc = 0; cc < COLS; ++cc) An[i][cc] = 0.0f;
#pragma unroll
                        for (int k = 0; k < N; ++k) {
                            const float m = REV ? Jr[k * N + i] : Jr[i * N + k];
                            bn[i] = fmaf(m, be[k], bn[i]);
#pragma unroll
                            for (int cc = 0; cc < COLS; ++cc) An[i][cc] = fmaf(m, A[k][cc], An[i][cc]);
                        }
                    }
#pragma unroll
                    for (int i = 0; i < N; ++i) {
                        be[i] = bn[i];
#pragma unroll
                        for (int cc = 0; cc < COLS; ++cc) A[i][cc] = An[i][cc];
                    }
                }
            }
            {
                float *ag = agg + chain * AGG;
#pragma unroll
                for (int i = 0; i < N; ++i) {
#pragma unroll
                    for (int cc = 0; cc < COLS; ++cc) ag[i * N + sub * COLS + cc] = A[i][cc];
                    if (sub == 0) ag[NN + i] = be[i];
                }
            }
            __syncwarp();
            // warp aggregate, then tile aggregate (warp 0), then publish
            {
                const float *first = agg + (warp * CPW) * AGG;
                float *t0 = tmp + warp * 2 * AGG, *t1 = t0 + AGG;
                const float *cur = first;
                for (int k = 1; k < CPW; ++k) {
                    float *dst = (k == CPW - 1) ? (wagg + warp * AGG) : ((k & 1) ? t0 : t1);
                    combine_smem<N>(dst, agg + (warp * CPW + k) * AGG, cur, lane);
                    cur = dst;
                }
                if (CPW == 1) {
                    for (int o = lane; o < AGG; o += 32) wagg[warp * AGG + o] = first[o];
                    __syncwarp();
                }
            }
            __syncthreads();
            if (warp == 0) {
                float *t0 = tmp, *t1 = tmp + AGG;
                const float *cur = wagg;
                for (int k = 1; k < WARPS; ++k) {
                    float *dst = (k == WARPS - 1) ? tagg : ((k & 1) ? t0 : t1);
                    combine_smem<N>(dst, wagg + k * AGG, cur, lane);
                    cur = dst;
                }
                float *g = w.aggs + tile_index * AGG;
                for (int o = lane; o < AGG; o += 32) g[o] = tagg[o];
                __threadfence();
                __syncwarp();
                if (lane == 0) st_release_u32(w.flags + tile_index, 1u);
            }
            continue;
        }

        // ------------------------------------------------ B item: states entering each warp, each chain
        if (warp == 0) {
            if (lane < N) wstart[lane] = ystart[lane];
            __syncwarp();
            for (int k = 0; k + 1 < WARPS; ++k)
                matvec_smem<N>(wstart + (k + 1) * N, wagg + k * AGG, wstart + k * N, lane);
        }
        __syncthreads();
        {
            float *cs = cstart + (warp * CPW) * N;
            if (lane < N) cs[lane] = wstart[warp * N + lane];
            __syncwarp();
            for (int k = 0; k + 1 < CPW; ++k)
                matvec_smem<N>(cs + (k + 1) * N, agg + (warp * CPW + k) * AGG, cs + k * N, lane);
        }

        // ------------------------------------------------ apply: replay the chain, y overwrites b
        if constexpr (N == 1) {
            float yv = cstart[chain];
#pragma unroll 1
            for (int q4 = 0; q4 < S / 4; ++q4) {
                if (4 * q4 >= cnt) break;
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
                *reinterpret_cast<float4 *>(sB + base) = b4;
            }
        } else {
            float y[N];
#pragma unroll
            for (int k = 0; k < N; ++k) y[k] = cstart[chain * N + k];
#pragma unroll 1
            for (int q = 0; q < cnt; ++q) {
                const bool ident = REV && (s0 + chain * S + q == 0);
                const float *Je = sJ + tg.j_off(chain, q, cnt);
                float *bv = sB + tg.b_off(chain, q, cnt);
                float v[COLS];
#pragma unroll
                for (int cc = 0; cc < COLS; ++cc) {
                    const int i = sub * COLS + cc;
                    float acc = bv[i];
                    if (ident) {
#pragma unroll
                        for (int k = 0; k < N; ++k) if (k == i) acc += y[k];
                    } else if (!REV) {
                        if constexpr (N >= 4) {
#pragma unroll
                            for (int v4 = 0; v4 < N / 4; ++v4) {
                                const float4 f = reinterpret_cast<const float4 *>(Je + i * N)[v4];
                                acc = fmaf(f.x, y[4 * v4], acc); acc = fmaf(f.y, y[4 * v4 + 1], acc);
                                acc = fmaf(f.z, y[4 * v4 + 2], acc); acc = fmaf(f.w, y[4 * v4 + 3], acc);
                            }
                        } else {
#pragma unroll
                            for (int k = 0; k < N; ++k) acc = fmaf(Je[i * N + k], y[k], acc);
                        }
                    } else {
#pragma unroll
                        for (int k = 0; k < N; ++k) acc = fmaf(Je[k * N + i], y[k], acc);
                    }
                    v[cc] = acc;
                }
#pragma unroll
                for (int cc = 0; cc < COLS; ++cc) bv[sub * COLS + cc] = v[cc];
#pragma unroll
                for (int k = 0; k < N; ++k) y[k] = __shfl_sync(chain_mask, v[k % COLS], chain_lane0 + k / COLS);
            }
        }
        __syncthreads();

        // ------------------------------------------------ stream y out (+ max |y - yold|)
        {
            const size_t gbase = ((size_t)seq * T + tg.t_lo()) * N;
            float *yo = a.y + gbase;
            const float *yold = a.yold ? a.yold + gbase : nullptr;
            const int total = Lt * N;
            const bool vec = (N >= 4 || (tg.dense_base() * N) % 4 == 0) && (((uintptr_t)yo & 15) == 0) &&
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
        if (lane == 0 && mb) atomicMax(&a.st->err_bits, mb);
    }
}

}  // namespace deer
