// Single-pass scan of the linear recurrence for n = 4 (Sec. 2.2 / Eq. 5 solve; App. B.1 adjoint).
//
// Same roles as the n <= 2 kernel (workers publish tile aggregates, resolver warps walk a
// sequence's aggregates in order and publish the state entering every tile, every wait bounded),
// with both directions of the exchange as 64-bit {value, flag} words (one round trip, no fence),
// and a worker CTA holds ONE tile at a time and visits it twice back to back:
//
//   stage the tile's J (per-thread 16-byte cp.async into run-padded shared memory); each thread
//   reads the b of its own chain straight from global memory into registers meanwhile
//   A: every thread folds its chain of S positions into (A, beta) in registers; a warp-shuffle
//      scan gives each thread its chain's exclusive prefix inside the warp, which STAYS IN
//      REGISTERS; warp 0 combines the warp aggregates and publishes the tile aggregate
//   warp 1 polls for the state entering the tile; once it is there the last thread claims the
//   CTA's next tile (the atomic's latency hides behind the replay)
//   B: every thread replays its chain from (warp prefix, chain prefix)(entering state); y_t goes
//      into the part of the chain's J run that the replay has already consumed and is streamed
//      out from there, coalesced, with the max |y - y_old| reduction
//
// The tile is read from HBM once and never staged twice; five CTA barriers per tile.  Shared
// memory per CTA is the tile's J plus a few hundred bytes (43 KB), so five CTAs share an SM.
#pragma once
#include "scan_onepass.cuh"

namespace deer {

// shared memory of a worker CTA: the tile's J, the warp prefixes and aggregates, the entering state
struct Hold4 {
    using C = OnePass<4>;
    static constexpr int SM_FLOATS = C::JBUF + C::PEND + C::WARPS * 2 * C::AGG + 4 + 4;
    static constexpr size_t SMEM = SM_FLOATS * sizeof(float) + 128;
    static_assert(32 * C::AGG <= C::JBUF / C::WARPS, "resolver staging must fit the tile buffer");
};

template <bool REV>
__global__ void __launch_bounds__(OnePass<4>::THREADS, 5) scan_hold4_kernel(ScanArgs a, OnePassWs w)
{
    constexpr int N = 4, NN = 16;
    using C = OnePass<N>;
    static_assert(C::HOLD && C::PADDED, "one tile per CTA, run-padded layout");
    constexpr int S = C::S, CHAINS = C::CHAINS, AGG = C::AGG, WARPS = C::WARPS, THREADS = C::THREADS;
    constexpr int PPE = NN / 4;                     // 16-byte pieces per J_t
    constexpr int CLAIMER = THREADS - 1;
    static_assert((C::L * PPE) % THREADS == 0 && C::L % THREADS == 0, "full-tile loops have constant trip counts");

    extern __shared__ __align__(16) float smem_raw[];
    float *sJ = (float *)(((uintptr_t)smem_raw + 127) & ~(uintptr_t)127);
    float *wagg = sJ + C::JBUF;                     // exclusive warp prefixes
    float *tmp = wagg + C::PEND;                    // warp aggregates
    float *ystart = tmp + WARPS * 2 * AGG;
    __shared__ int s_seq, s_c, s_abort, s_role, s_done;

    pdl_prologue();
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const int chain = tid;
    const int T = a.T;

    // the role ticket and the loop-ended word travel together (one round trip; a ticket taken by a
    // launch that then returns is harmless: the counters are rewound before the next evaluation)
    if (tid == 0) {
        const unsigned ticket = atomicAdd(&a.st->role_counter, 1u);
        s_done = loop_ended(a.st) ? 1 : 0;
        s_abort = 0;
        s_role = (int)ticket;
    }
    __syncthreads();
    if (s_done) return;
    if (s_role < w.resolvers) {
        resolver_ll_loop<N>(a, w, sJ, s_role * WARPS + warp, w.resolvers * WARPS, lane);
        __syncthreads();
        if (tid == 0) scan_epilogue(a.st);
        return;
    }
    unsigned mb = 0;          // running max |y - yold| bits of this thread

    // claim: tile ids come from the same counter as the role tickets (ticket - resolvers), so a
    // worker's ticket is its first tile id (no second atomic before the first tile) and ids are still
    // handed out in order to running CTAs only; id -> (seq, tile), padding ids of the last window are
    // skipped; c < 0 when no tile is left
    auto next_ticket = [&]() { return atomicAdd(&a.st->role_counter, 1u) - (unsigned)w.resolvers; };
    auto claim_from = [&](unsigned id, int &seq, int &c) {
        for (;;) {
            if (id >= w.total_ids) { c = -1; return; }
            const unsigned j = id % (unsigned)w.Wd;
            const unsigned ws_ = id / (unsigned)w.Wd;
            seq = (int)(ws_ % (unsigned)a.B);
            const unsigned win = ws_ / (unsigned)a.B;
            c = (int)(win * (unsigned)w.Wd + j);
            if (c < w.nch) return;
            id = next_ticket();
        }
    };
    // geometry and sources of one tile
    struct Tile {
        TileGeom<N, REV> tg;
        const float *Jsrc, *bsrc;
        size_t index, gbase;
        int jcnt;
        bool full;      // all runs complete and every J_t present: each chain's run is one contiguous
                        // block of S positions in global memory and offsets follow by constants
    };
    auto make_tile = [&](int seq, int c) {
        Tile t;
        t.tg.s0 = c * C::L;
        t.tg.Lt = min(C::L, T - t.tg.s0);
        t.tg.T = T;
        const size_t p_lo = t.tg.t_lo();                                   // first b element of the tile
        const size_t j_lo = REV ? p_lo + 1 : p_lo;                         // first J element of the tile
        t.jcnt = (REV && t.tg.s0 == 0) ? t.tg.Lt - 1 : t.tg.Lt;            // (reverse: J[T] does not exist)
        t.index = (size_t)seq * w.nch + c;
        t.Jsrc = a.J + ((size_t)seq * T + j_lo) * NN;
        t.gbase = ((size_t)seq * T + p_lo) * N;
        t.bsrc = a.b + t.gbase;
        t.full = t.tg.Lt == C::L && t.jcnt == C::L;
        return t;
    };
    // float offset inside a chain's J run of the y of local index li (ascending t within the run)
    // when the run holds cnt positions: always inside matrices the replay has consumed by then
    // (forward: the run's first floats; reverse: its last ones, as the replay walks down the run)
    auto y_slot = [](int cnt, int li) { return REV ? 12 * cnt + 4 * li : 4 * li; };
    auto full_off = [&](int u) {        // float offset into sJ of the y of ascending-t position u of a full tile
        const int blk = u / S, within = u - blk * S;
        return (REV ? CHAINS - 1 - blk : blk) * C::JRUN + (REV ? 12 * S : 0) + 4 * within;
    };
    auto any_off = [&](const TileGeom<N, REV> &tg, int u) {     // the same for any tile
        int r, li;
        tg.locate(u, r, li);
        return r * C::JRUN + y_slot(tg.run_cnt(r), li);
    };
    auto stage_J = [&](const Tile &t) {
        if (t.full) {
            constexpr int RUN_PIECES = S * PPE;
#pragma unroll
            for (int k = 0; k < C::L * PPE / THREADS; ++k) {
                const int p = tid + k * THREADS;
                const int blk = p / RUN_PIECES, within = p - blk * RUN_PIECES;
                cp_async16(sJ + (REV ? CHAINS - 1 - blk : blk) * C::JRUN + within * 4, t.Jsrc + (size_t)p * 4);
            }
        } else {
            for (int g = tid; g < t.jcnt * PPE; g += THREADS) {
                const int u = g / PPE, v = g - u * PPE;
                cp_async16(sJ + t.tg.jmat_off(u) + v * 4, t.Jsrc + (size_t)u * NN + v * 4);
            }
        }
        cp_async_commit();
    };
    // b of this thread's chain by scan step q (scan offset chain*S + q of the tile <-> ascending-t
    // index chain*S + q forward, Lt - 1 - (chain*S + q) reverse); zeros beyond the run
    auto load_b = [&](const Tile &t, int cnt, float4 (&bs)[S]) {
        const float4 *src = reinterpret_cast<const float4 *>(t.bsrc);
#pragma unroll
        for (int q = 0; q < S; ++q) {
            const int u = REV ? t.tg.Lt - 1 - (S * chain + q) : S * chain + q;
            bs[q] = (q < cnt) ? __ldg(src + u) : make_float4(0.0f, 0.0f, 0.0f, 0.0f);
        }
    };
    // one step of the chain from the staged tile: M = J (forward) or J^T (reverse; identity at scan position 0)
    auto load_M = [&](const TileGeom<N, REV> &tg, int q, int cnt, float (&M)[N][N]) {
        const float *Je = sJ + tg.j_off(chain, q, cnt);
        float R[4][4];
#pragma unroll
        for (int i = 0; i < 4; ++i) {
            const float4 f = reinterpret_cast<const float4 *>(Je)[i];
            R[i][0] = f.x; R[i][1] = f.y; R[i][2] = f.z; R[i][3] = f.w;
        }
        const bool ident = REV && (tg.s0 + chain * S + q == 0);
#pragma unroll
        for (int i = 0; i < 4; ++i)
#pragma unroll
            for (int k = 0; k < 4; ++k) M[i][k] = ident ? ((i == k) ? 1.0f : 0.0f) : (REV ? R[k][i] : R[i][k]);
    };

    if (tid == CLAIMER) {
        int seq = -1, c = -1;
        claim_from((unsigned)(s_role - w.resolvers), seq, c);
        s_seq = seq; s_c = c;
    }
    __syncthreads();
    int seq = s_seq, c = s_c;
    while (c >= 0) {
        const Tile t = make_tile(seq, c);
        const TileGeom<N, REV> &tg = t.tg;
        const int cnt = tg.run_cnt(chain);
        stage_J(t);
        float4 bs[S];
        load_b(t, cnt, bs);   // in flight together with the J copies
        cp_async_wait_0();
        __syncthreads();      // tile staged; every thread has read s_seq / s_c

        // ------------------------------------------------ A: chain aggregates, prefixes, publish
        RegAgg<N> held;       // this chain's exclusive prefix inside the warp
        {
            RegAgg<N> r;
            ragg_identity<N>(r);
#pragma unroll
            for (int q = 0; q < S; ++q) {
                if (q < cnt) {
                    float M[N][N];
                    load_M(tg, q, cnt, M);
                    const float bq[N] = {bs[q].x, bs[q].y, bs[q].z, bs[q].w};
                    ragg_push<N>(r, M, bq);
                }
            }
            ragg_warp_scan<N>(r, held, lane);
            if (lane == 31) ragg_store<N>(tmp + warp * AGG, r);   // warp aggregate
        }
        __syncthreads();
        if (warp == 0) {
            RegAgg<N> wr, wex;
            if (lane < WARPS) ragg_load<N>(wr, tmp + lane * AGG);
            else ragg_identity<N>(wr);
            ragg_warp_scan<N, WARPS>(wr, wex, lane);
            if (lane == WARPS - 1) {
                // tile aggregate as {value, flag} words: no fence, and one round trip for the reader
                unsigned long long *dst = reinterpret_cast<unsigned long long *>(w.aggs) + t.index * AGG;
#pragma unroll
                for (int i = 0; i < N; ++i) {
#pragma unroll
                    for (int j = 0; j < N; ++j)
                        st_relaxed_u64(dst + i * N + j, LL_FLAG | (unsigned long long)__float_as_uint(wr.A[i][j]));
                    st_relaxed_u64(dst + N * N + i, LL_FLAG | (unsigned long long)__float_as_uint(wr.be[i]));
                }
            }
            if (lane < WARPS) ragg_store<N>(wagg + lane * AGG, wex);   // exclusive prefix over warps
        } else if (warp == 1) {
            // the state entering the tile ({value, flag} words written by the sequence's resolver)
            const unsigned long long *src = w.starts + t.index * N;
            unsigned spins = 0;
            bool ok = true;
            for (;;) {
                const unsigned long long v = (lane < N) ? ld_relaxed_u64(src + lane) : LL_FLAG;
                if (__all_sync(0xffffffffu, v != 0ull)) {
                    if (lane < N) {
                        ystart[lane] = __uint_as_float((unsigned)(v & 0xffffffffull));
                        st_relaxed_u64(w.starts + t.index * N + lane, 0ull);     // consumed: cleared for the next launch
                    }
                    break;
                }
                if (!keep_spinning(a, spins)) { ok = false; break; }
            }
            if (!__all_sync(0xffffffffu, ok)) s_abort = 1;
        }
        __syncthreads();      // ystart, warp prefixes and s_abort visible
        if (s_abort) break;
        // the CTA's next tile is claimed only now, when nothing this CTA still has to do depends on
        // another CTA (a tile claimed earlier would sit unstarted while the sequence's chain waits
        // for its aggregate); the atomic's latency hides behind the replay
        unsigned next_id = 0;
        if (tid == CLAIMER) next_id = next_ticket();

        // ------------------------------------------------ B: replay from the entering state
        {
            if constexpr (REV) load_b(t, cnt, bs);      // (reverse: read again rather than kept in registers)
            float y[N];
#pragma unroll
            for (int k = 0; k < N; ++k) y[k] = ystart[k];
            RegAgg<N> e;
            ragg_load<N>(e, wagg + warp * AGG);
            ragg_apply<N>(e, y);
            ragg_apply<N>(held, y);
#pragma unroll
            for (int q = 0; q < S; ++q) {
                if (q < cnt) {
                    float M[N][N];
                    load_M(tg, q, cnt, M);
                    const float bq[N] = {bs[q].x, bs[q].y, bs[q].z, bs[q].w};
                    float yn[N];
#pragma unroll
                    for (int i = 0; i < N; ++i) {
                        yn[i] = bq[i];
#pragma unroll
                        for (int k = 0; k < N; ++k) yn[i] = fmaf(M[i][k], y[k], yn[i]);
                    }
#pragma unroll
                    for (int i = 0; i < N; ++i) y[i] = yn[i];
                    // into the part of the run that is already consumed (local index of step q: q forward, cnt-1-q reverse)
                    *reinterpret_cast<float4 *>(sJ + chain * C::JRUN + y_slot(cnt, REV ? cnt - 1 - q : q)) =
                        make_float4(yn[0], yn[1], yn[2], yn[3]);
                }
            }
        }
        if (tid == CLAIMER) {
            int ns = -1, nc_ = -1;
            claim_from(next_id, ns, nc_);
            s_seq = ns; s_c = nc_;
        }
        __syncthreads();      // y complete in shared memory; next tile known
        const int nseq = s_seq, nc = s_c;

        // ------------------------------------------------ stream y out (+ max |y - yold|)
        {
            float *yo = a.y + t.gbase;
            const float *yold = a.yold ? a.yold + t.gbase : nullptr;
            const bool vec = (((uintptr_t)yo & 15) == 0) && (!yold || ((uintptr_t)yold & 15) == 0);
            auto put = [&](int u, int off) {
                const float4 val = *reinterpret_cast<const float4 *>(sJ + off);
                if (yold) {
                    const float4 o = __ldg(reinterpret_cast<const float4 *>(yold) + u);
                    mb = max(mb, absdiff_bits(val.x, o.x)); mb = max(mb, absdiff_bits(val.y, o.y));
                    mb = max(mb, absdiff_bits(val.z, o.z)); mb = max(mb, absdiff_bits(val.w, o.w));
                }
                reinterpret_cast<float4 *>(yo)[u] = val;
            };
            if (vec && t.full) {
#pragma unroll
                for (int k = 0; k < C::L / THREADS; ++k) put(tid + k * THREADS, full_off(tid + k * THREADS));
            } else if (vec) {
                for (int u = tid; u < tg.Lt; u += THREADS) put(u, any_off(tg, u));
            } else {
                for (int g = tid; g < tg.Lt * N; g += THREADS) {
                    const float val = sJ[any_off(tg, g / N) + g % N];
                    if (yold) mb = max(mb, absdiff_bits(val, yold[g]));
                    yo[g] = val;
                }
            }
        }
        __syncthreads();      // the tile buffer is free
        seq = nseq; c = nc;
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
