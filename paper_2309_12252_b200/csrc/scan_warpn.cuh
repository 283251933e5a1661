// Single-pass scan for n = 16 and n = 32: one warp per chain, chain product on tensor cores.
//
// The n = 8 design of scan_warp8.cuh with the n x n running product tiled into m16n8k8 fragments:
//   * the warp keeps X = P^T (n x n) in (n/16) x (n/8) accumulator fragments and advances it with
//         X <- X * M,   M = J_t^T (forward)  or  J_{t+1} (reverse),
//     as (n/16)(n/8)(n/8) MMAs per position, each issued three times on hi/lo TF32 splits; the
//     accumulator fragment of column block kk is the A operand of contraction block kk (the same
//     renaming of the contraction index as for n = 8), and the B operand of (kk, nn) is the lane's
//     8-byte piece J[8nn+g][8kk+2t .. +1] (forward) or the scalars J[8kk+2t][8nn+g], J[8kk+2t+1][8nn+g]
//     (reverse);
//   * the matrices and vectors of a chain stream through a warp-private shared-memory ring filled
//     with 16-byte cp.async copies (no registers held while loads are in flight, only __syncwarp
//     between stages); rows are padded so that the operand reads of either direction are free
//     of bank conflicts;
//   * beta is carried as a separate mat-vec chain started from zero (the same routine replays the
//     chain from its true entering state in the B item): lane (g,t) holds y[8kk+2t], y[8kk+2t+1];
//   * warp aggregates are combined by warp 0 with the same step, reading them from shared memory.
// Tiles, items, resolvers, flags and bounded waits are those of scan_onepass.cuh.
#pragma once
#include "scan_warp8.cuh"

namespace deer {

template <int N> struct WarpN {
    static constexpr int NN = N * N, AGG = N * N + N;
    static constexpr int NT = N / 8;                   // 8-wide column / contraction blocks
    static constexpr int MT = N / 16;                  // 16-high row blocks of X
    static constexpr int WARPS = (N == 16) ? 8 : 4;    // chains per tile
    static constexpr int THREADS = WARPS * 32;
    static constexpr int SW_MIN = 16, SW_MAX = 64;     // positions per warp chain (chosen per problem size)
    static constexpr int CTAS_PER_SM = 3;
    // longest chain that still leaves about 1.5 tiles per resident CTA (see Warp8::chain_len)
    static int chain_len(int B, int T, int resident_ctas)
    {
        int sw = SW_MAX;
        while (sw > SW_MIN && (long long)B * ((T + WARPS * sw - 1) / (WARPS * sw)) < 3LL * resident_ctas / 2) sw >>= 1;
        return sw;
    }
    static constexpr int Q = 2;                        // pending tiles per CTA
    static constexpr int STAGES = (N == 16) ? 4 : 2;   // ring depth per warp (positions)
    static constexpr int STAGE_FLOATS = N * (N + 8) + N;   // matrix with padded rows, then the vector
    static constexpr int RES_WARPS = 4;                // warps of a resolver CTA that resolve, at most (see big_res_warps)
    static constexpr int RES_SLOTS = (N == 16) ? 64 : 16; // tile aggregates a resolver CTA stages, shared by its resolving warps
    static constexpr int PEND = (WARPS - 1) * AGG;     // warp aggregates kept for the B item (the last warp's
                                                       // is only needed by the tile combine: it sits in that warp's ring)
    static constexpr int SM_WORK = Q * PEND + WARPS * N + N + 16 + WARPS * STAGES * STAGE_FLOATS;
    static constexpr int SM_RES = RES_SLOTS * AGG + RES_WARPS * N;   // tile slots, then a state vector per resolving warp
    static constexpr int SM_FLOATS = SM_WORK > SM_RES ? SM_WORK : SM_RES;
    static constexpr size_t SMEM = SM_FLOATS * sizeof(float) + 128;
    static constexpr int MAX_SEQ_PER_WARP = 8;
    static_assert(N == 16 || N == 32, "one row of the state per resolver lane");
};

// Resolver for n in {16, 32}: a warp walks Y <- A Y + beta over the published tile aggregates of its sequences and
// writes the state entering every tile (lane i holds component i of the running state).  The walk over a sequence's
// tiles is the serial part of a scan, so the memory round trips are kept off it: a warp that serves ONE sequence
// (batches up to the resolver warp count) keeps two batches of aggregates in shared memory, fetched by asynchronous
// copies once their flags have been seen (a ring of tile slots, up to four fetch groups in flight), so that the flags
// of the tiles after next and the bytes of the next tiles travel while the current ones are walked.  The fewer
// sequences a launch has, the fewer warps of a resolver CTA resolve and the deeper each one's ring (big_res_warps).  A warp with several sequences visits them in turn (one batch per visit,
// all of its bytes in flight at once).
template <int N>
__device__ __forceinline__ void resolver_big_fetch(float *dst, const float *src, int cnt, int lane)
{
    constexpr int AGG = WarpN<N>::AGG;
    const int total4 = cnt * AGG / 4;
    for (int i = lane; i < total4; i += 32) cp_async16(dst + 4 * i, src + 4 * i);
    cp_async_commit();
}

// the walk over `cnt` staged aggregates; out: the tiles' entering-state words.  Lane i owns component i of the state
// and row i of A; the state goes through a vector in shared memory (ybuf) so that a row and the state are read as
// 16-byte pieces -- 2 x n/4 loads and n FMAs per tile where a shuffle per element took three times the instructions --
// each lane starting at a different piece (the eight lanes of a 128-bit access phase then hit distinct banks).
template <int N>
__device__ __forceinline__ float resolver_big_walk(const float *stage, int cnt, unsigned long long *out, float y, float *ybuf, int lane)
{
    constexpr int AGG = WarpN<N>::AGG, NN = WarpN<N>::NN, CH = N / 4;
    const int sw = (N == 32) ? (lane & 7) : ((lane >> 1) & 3);
    const int rl = lane < N ? lane : 0;
    const float4 *yb = reinterpret_cast<const float4 *>(ybuf);
    for (int q = 0; q < cnt; ++q) {
        if (lane < N) {
            st_relaxed_u64(out + q * N + lane, LL_FLAG | (unsigned long long)__float_as_uint(y));
            ybuf[lane] = y;
        }
        __syncwarp();
        const float *ag = stage + q * AGG;
        const float4 *row = reinterpret_cast<const float4 *>(ag + rl * N);
        float a0 = (lane < N) ? ag[NN + lane] : 0.0f, a1 = 0.0f, a2 = 0.0f, a3 = 0.0f;
#pragma unroll
        for (int k = 0; k < CH; ++k) {
            const int kk = k ^ sw;
            const float4 av = row[kk], yv = yb[kk];
            a0 = fmaf(av.x, yv.x, a0); a1 = fmaf(av.y, yv.y, a1);
            a2 = fmaf(av.z, yv.z, a2); a3 = fmaf(av.w, yv.w, a3);
        }
        y = (a0 + a1) + (a2 + a3);
        __syncwarp();              // every lane has read the state before the next tile's is written
    }
    return y;
}

template <int N>
__device__ void resolver_big(const ScanArgs &a, const OnePassWs &w, float *stage_all, int rw, int nrw, int lane)
{
    if (a.no_resolve) return;     // (wait-expiry test: nobody publishes entering states)
    using C = WarpN<N>;
    constexpr int AGG = C::AGG;
    const int RING = C::RES_SLOTS / w.res_warps;                           // this warp's tile slots (a power of two)
    float *stage = stage_all + (threadIdx.x >> 5) * RING * AGG;
    float *ybuf = stage_all + C::RES_SLOTS * AGG + (threadIdx.x >> 5) * N;
    unsigned spins = 0;
    if (rw + nrw >= a.B) {
        // ---- one sequence: a ring of RING tile slots, up to four fetch groups in flight
        const int s = rw;
        if (s >= a.B) return;
        const unsigned *flags = w.flags + (size_t)s * w.nch;
        const float *aggs = w.aggs + (size_t)s * w.nch * AGG;
        unsigned long long *starts = w.starts + (size_t)s * w.nch * N;
        float y = (lane < N && a.y0) ? a.y0[(size_t)s * N + lane] : 0.0f;
        int c = 0, f = 0;                      // next tile to walk, next tile to fetch (tile i sits in slot i % RING)
        int ng = 0, ghead = 0, gcnt[4] = {0, 0, 0, 0};
        unsigned fl = (lane < w.nch) ? ld_acquire_u32(flags + lane) : 0u;      // flags of tiles f + lane
        while (c < w.nch) {
            bool progressed = false;
            if (ng < 4 && f < w.nch && f - c < RING) {
                const unsigned m = __ballot_sync(0xffffffffu, fl >= 1u);
                __syncwarp();      // orders every lane's aggregate copies below after the acquiring lanes' flag loads
                int r = (m == 0xffffffffu) ? 32 : (__ffs(~m) - 1);
                r = min(r, RING - (f - c));            // (all free slots at once: measured better than smaller groups)
                if (r > 0) {
                    // tiles f .. f+r-1 into their slots (the range may wrap around the ring): one group
                    const int s0 = f & (RING - 1), first = min(r, RING - s0);
                    const int n4a = first * AGG / 4, n4b = (r - first) * AGG / 4;
                    const float *src = aggs + (size_t)f * AGG;
                    for (int i = lane; i < n4a; i += 32) cp_async16(stage + s0 * AGG + 4 * i, src + 4 * i);
                    for (int i = lane; i < n4b; i += 32) cp_async16(stage + 4 * i, src + first * AGG + 4 * i);
                    cp_async_commit();
                    gcnt[(ghead + ng) & 3] = r;
                    f += r;
                    ++ng;
                    progressed = true;
                }
                fl = (f + lane < w.nch) ? ld_acquire_u32(flags + f + lane) : 0u;
            }
            if (ng > 0) {
                if (ng == 1) cp_async_wait_0(); else if (ng == 2) cp_async_wait_1(); else if (ng == 3) cp_async_wait_2(); else cp_async_wait_3();
                __syncwarp();
                const int cnt = gcnt[ghead];
                const int s0 = c & (RING - 1), first = min(cnt, RING - s0);
                y = resolver_big_walk<N>(stage + s0 * AGG, first, starts + (size_t)c * N, y, ybuf, lane);
                if (cnt > first) y = resolver_big_walk<N>(stage, cnt - first, starts + (size_t)(c + first) * N, y, ybuf, lane);
                __syncwarp();
                if (lane < cnt) w.flags[(size_t)s * w.nch + c + lane] = 0u;   // consumed: cleared for the next launch
                c += cnt;
                ghead = (ghead + 1) & 3;
                --ng;
                progressed = true;
            }
            if (progressed) spins = 0;
            else if (!keep_spinning(a, spins)) { cp_async_wait_0(); return; }
        }
        return;
    }
    // ---- several sequences per warp
    int nseq = 0;
    int pos[C::MAX_SEQ_PER_WARP];
    float yv[C::MAX_SEQ_PER_WARP];
    unsigned fnext[C::MAX_SEQ_PER_WARP];
#pragma unroll
    for (int k = 0; k < C::MAX_SEQ_PER_WARP; ++k) {
        pos[k] = 0; yv[k] = 0.0f; fnext[k] = 0u;
        const int s = rw + k * nrw;
        if (s < a.B) {
            nseq = k + 1;
            if (lane < N && a.y0) yv[k] = a.y0[(size_t)s * N + lane];
            if (lane < w.nch) fnext[k] = ld_acquire_u32(w.flags + (size_t)s * w.nch + lane);
        }
    }
    int remaining = nseq;
    while (remaining > 0) {
        bool progressed = false;
#pragma unroll
        for (int k = 0; k < C::MAX_SEQ_PER_WARP; ++k) {
            if (k >= nseq) break;
            const int c0 = pos[k];
            if (c0 >= w.nch) continue;
            const int s = rw + k * nrw;
            const unsigned *flags = w.flags + (size_t)s * w.nch;
            const unsigned m = __ballot_sync(0xffffffffu, fnext[k] >= 1u);
            __syncwarp();      // orders every lane's aggregate copies below after the acquiring lanes' flag loads
            int cnt = (m == 0xffffffffu) ? 32 : (__ffs(~m) - 1);
            if (cnt > RING) cnt = RING;
            {
                const int j = c0 + cnt + lane;
                fnext[k] = (j < w.nch) ? ld_acquire_u32(flags + j) : 0u;
            }
            if (cnt == 0) continue;
            progressed = true;
            resolver_big_fetch<N>(stage, w.aggs + ((size_t)s * w.nch + c0) * AGG, cnt, lane);
            cp_async_wait_0();
            __syncwarp();
            yv[k] = resolver_big_walk<N>(stage, cnt, w.starts + ((size_t)s * w.nch + c0) * N, yv[k], ybuf, lane);
            __syncwarp();
            if (lane < cnt) w.flags[(size_t)s * w.nch + c0 + lane] = 0u;   // consumed: cleared for the next launch
            pos[k] = c0 + cnt;
            if (pos[k] >= w.nch) --remaining;
        }
        if (progressed) spins = 0;
        else if (!keep_spinning(a, spins)) return;
    }
}

// Row stride (floats) of a matrix in a ring stage.  Rows are padded so that the operand reads are
// free of bank conflicts with plain constant offsets: the forward operand reads 8-byte pieces of
// 4 rows x 4 columns per half-warp (stride = 8 mod 32 words), the reverse operand scalars of
// 4 rows (two apart) x 8 columns per warp (stride = 4 mod 16 words).
template <int N, bool REV> struct RingRow { static constexpr int RS = N + (REV ? 4 : 8); };

template <int K> __device__ __forceinline__ void cp_async_wait_n() { asm volatile("cp.async.wait_group %0;" ::"n"(K) : "memory"); }

// One position into a ring stage: the matrix (identity when `ident`) with padded rows, then the vector.
// Always commits one group, so the group count follows the position count.
template <int N, bool REV>
__device__ __forceinline__ void issue_stage_n(float *dst, const float *Jt, const float *bt, bool valid, bool ident, int lane)
{
    constexpr int NN = N * N, RS = RingRow<N, REV>::RS;
    if (valid) {
        if (ident) {
            for (int j = lane; j < NN / 4; j += 32) {
                const int row = j / (N / 4), ch = j % (N / 4);
                float4 v = make_float4(0.f, 0.f, 0.f, 0.f);
                if ((row >> 2) == ch) {
                    if ((row & 3) == 0) v.x = 1.0f;
                    if ((row & 3) == 1) v.y = 1.0f;
                    if ((row & 3) == 2) v.z = 1.0f;
                    if ((row & 3) == 3) v.w = 1.0f;
                }
                *reinterpret_cast<float4 *>(dst + row * RS + 4 * ch) = v;
            }
        } else {
#pragma unroll
            for (int u = 0; u < NN / 4 / 32; ++u) {
                const int j = lane + 32 * u;
                cp_async16(dst + (j / (N / 4)) * RS + 4 * (j % (N / 4)), Jt + 4 * j);
            }
        }
        if (lane < N / 4) cp_async16(dst + N * RS + 4 * lane, bt + 4 * lane);
    }
    cp_async_commit();
}

// The lane's pieces of one position's matrix from its ring stage,
// jp[nn][kk] = {M[8kk+2t][8nn+g], M[8kk+2t+1][8nn+g]}: forward M = J^T, reverse M = J.
template <int N, bool REV>
__device__ __forceinline__ void load_pieces(float (&jp)[N / 8][N / 8][2], const float *Ms, int g, int t)
{
    constexpr int NT = N / 8, RS = RingRow<N, REV>::RS;
    const float *base = REV ? Ms + (2 * t) * RS + g : Ms + g * RS + 2 * t;
#pragma unroll
    for (int nn = 0; nn < NT; ++nn)
#pragma unroll
        for (int kk = 0; kk < NT; ++kk) {
            if (!REV) {
                const float2 f = *reinterpret_cast<const float2 *>(base + 8 * nn * RS + 8 * kk);
                jp[nn][kk][0] = f.x; jp[nn][kk][1] = f.y;
            } else {
                jp[nn][kk][0] = base[8 * kk * RS + 8 * nn];
                jp[nn][kk][1] = base[8 * kk * RS + RS + 8 * nn];
            }
        }
}

// the same pieces of an aggregate (A row-major in shared memory; always the forward form)
template <int N>
__device__ __forceinline__ void load_pieces_smem(float (&jp)[N / 8][N / 8][2], const float *A, int g, int t)
{
    constexpr int NT = N / 8;
#pragma unroll
    for (int nn = 0; nn < NT; ++nn)
#pragma unroll
        for (int kk = 0; kk < NT; ++kk) {
            const float2 f = *reinterpret_cast<const float2 *>(A + (8 * nn + g) * N + 8 * kk + 2 * t);
            jp[nn][kk][0] = f.x; jp[nn][kk][1] = f.y;
        }
}

// X <- X * M on accumulator fragments acc[mm][nn] (row block mm, column block nn), 3 x TF32
template <int N>
__device__ __forceinline__ void chain_step_n(float (&acc)[N / 16][N / 8][4], const float (&jp)[N / 8][N / 8][2])
{
    constexpr int NT = N / 8, MT = N / 16;
    float nacc[MT][NT][4];
#pragma unroll
    for (int mm = 0; mm < MT; ++mm)
#pragma unroll
        for (int nn = 0; nn < NT; ++nn)
#pragma unroll
            for (int i = 0; i < 4; ++i) nacc[mm][nn][i] = 0.0f;
#pragma unroll
    for (int kk = 0; kk < NT; ++kk) {
        unsigned ah[MT][4], al[MT][4];
#pragma unroll
        for (int mm = 0; mm < MT; ++mm) {
            split_tf32(acc[mm][kk][0], ah[mm][0], al[mm][0]);
            split_tf32(acc[mm][kk][2], ah[mm][1], al[mm][1]);
            split_tf32(acc[mm][kk][1], ah[mm][2], al[mm][2]);
            split_tf32(acc[mm][kk][3], ah[mm][3], al[mm][3]);
        }
#pragma unroll
        for (int nn = 0; nn < NT; ++nn) {
            unsigned bh[2], bl[2];
            split_tf32(jp[nn][kk][0], bh[0], bl[0]);
            split_tf32(jp[nn][kk][1], bh[1], bl[1]);
#pragma unroll
            for (int mm = 0; mm < MT; ++mm) {
                mma_tf32(nacc[mm][nn], al[mm], bh, nacc[mm][nn]);
                mma_tf32(nacc[mm][nn], ah[mm], bl, nacc[mm][nn]);
                mma_tf32(nacc[mm][nn], ah[mm], bh, nacc[mm][nn]);
            }
        }
    }
#pragma unroll
    for (int mm = 0; mm < MT; ++mm)
#pragma unroll
        for (int nn = 0; nn < NT; ++nn)
#pragma unroll
            for (int i = 0; i < 4; ++i) acc[mm][nn][i] = nacc[mm][nn][i];
}

// X <- X * M with ONE TF32 product per tile (operands truncated to 10 mantissa bits by the tensor core, fp32
// accumulate: relative error about 1e-3).  Only for the Newton-update form of the iteration, whose fixed
// point does not depend on the accuracy of the linear solve.
template <int N>
__device__ __forceinline__ void chain_step_n1(float (&acc)[N / 16][N / 8][4], const float (&jp)[N / 8][N / 8][2])
{
    constexpr int NT = N / 8, MT = N / 16;
    float nacc[MT][NT][4];
#pragma unroll
    for (int mm = 0; mm < MT; ++mm)
#pragma unroll
        for (int nn = 0; nn < NT; ++nn)
#pragma unroll
            for (int i = 0; i < 4; ++i) nacc[mm][nn][i] = 0.0f;
#pragma unroll
    for (int kk = 0; kk < NT; ++kk) {
        unsigned af[MT][4];
#pragma unroll
        for (int mm = 0; mm < MT; ++mm) {
            af[mm][0] = __float_as_uint(acc[mm][kk][0]);
            af[mm][1] = __float_as_uint(acc[mm][kk][2]);
            af[mm][2] = __float_as_uint(acc[mm][kk][1]);
            af[mm][3] = __float_as_uint(acc[mm][kk][3]);
        }
#pragma unroll
        for (int nn = 0; nn < NT; ++nn) {
            const unsigned bf[2] = {__float_as_uint(jp[nn][kk][0]), __float_as_uint(jp[nn][kk][1])};
#pragma unroll
            for (int mm = 0; mm < MT; ++mm) mma_tf32(nacc[mm][nn], af[mm], bf, nacc[mm][nn]);
        }
    }
#pragma unroll
    for (int mm = 0; mm < MT; ++mm)
#pragma unroll
        for (int nn = 0; nn < NT; ++nn)
#pragma unroll
            for (int i = 0; i < 4; ++i) acc[mm][nn][i] = nacc[mm][nn][i];
}

// y <- M^T-form mat-vec: ynew[nn] = y_new[8nn+g] (in the 4 lanes of group g); yv[kk] = {y[8kk+2t], y[8kk+2t+1]}
template <int N>
__device__ __forceinline__ void matvec_step(float (&yv)[N / 8][2], const float (&jp)[N / 8][N / 8][2],
                                            const float (&bg)[N / 8], float (&ynew)[N / 8], int t)
{
    constexpr int NT = N / 8;
#pragma unroll
    for (int nn = 0; nn < NT; ++nn) {
        float2 p2 = make_float2(0.0f, 0.0f);
#pragma unroll
        for (int kk = 0; kk < NT; ++kk)
            p2 = ffma2(make_float2(jp[nn][kk][0], jp[nn][kk][1]), make_float2(yv[kk][0], yv[kk][1]), p2);
        float part = p2.x + p2.y;
        part += __shfl_xor_sync(0xffffffffu, part, 1);
        part += __shfl_xor_sync(0xffffffffu, part, 2);
        ynew[nn] = part + bg[nn];
    }
#pragma unroll
    for (int kk = 0; kk < NT; ++kk) {
        yv[kk][0] = __shfl_sync(0xffffffffu, ynew[kk], 4 * (2 * t));
        yv[kk][1] = __shfl_sync(0xffffffffu, ynew[kk], 4 * (2 * t + 1));
    }
}

// X = P^T in fragments  ->  P row-major (+ beta from the distributed vector) at dst (shared or global)
template <int N>
__device__ __forceinline__ void store_aggregate(float *dst, const float (&acc)[N / 16][N / 8][4],
                                                const float (&yv)[N / 8][2], int g, int t)
{
    constexpr int NT = N / 8, MT = N / 16, NN = N * N;
#pragma unroll
    for (int mm = 0; mm < MT; ++mm)
#pragma unroll
        for (int nn = 0; nn < NT; ++nn) {
            const int r = 16 * mm + g, c = 8 * nn + 2 * t;      // X[r][c] = P[c][r]
            dst[c * N + r] = acc[mm][nn][0];
            dst[(c + 1) * N + r] = acc[mm][nn][1];
            dst[c * N + r + 8] = acc[mm][nn][2];
            dst[(c + 1) * N + r + 8] = acc[mm][nn][3];
        }
    if (g == 0) {
#pragma unroll
        for (int kk = 0; kk < NT; ++kk) {
            dst[NN + 8 * kk + 2 * t] = yv[kk][0];
            dst[NN + 8 * kk + 2 * t + 1] = yv[kk][1];
        }
    }
}

template <int N>
__device__ __forceinline__ void identity_fragments(float (&acc)[N / 16][N / 8][4], int g, int t)
{
#pragma unroll
    for (int mm = 0; mm < N / 16; ++mm)
#pragma unroll
        for (int nn = 0; nn < N / 8; ++nn) {
            const int r = 16 * mm + g, c = 8 * nn + 2 * t;
            acc[mm][nn][0] = (r == c) ? 1.0f : 0.0f;
            acc[mm][nn][1] = (r == c + 1) ? 1.0f : 0.0f;
            acc[mm][nn][2] = (r + 8 == c) ? 1.0f : 0.0f;
            acc[mm][nn][3] = (r + 8 == c + 1) ? 1.0f : 0.0f;
        }
}

template <int N, bool REV>
__global__ void __launch_bounds__(WarpN<N>::THREADS, WarpN<N>::CTAS_PER_SM) scan_warpn_kernel(ScanArgs a, OnePassWs w)
{
    using C = WarpN<N>;
    constexpr int NN = C::NN, AGG = C::AGG, NT = C::NT, MT = C::MT, WARPS = C::WARPS, Q = C::Q;
    pdl_prologue();
    if (loop_ended(a.st)) return;

    extern __shared__ __align__(16) float smem_raw[];
    float *sm = (float *)(((uintptr_t)smem_raw + 127) & ~(uintptr_t)127);
    float *pend = sm;                          // Q x warp aggregates (A row-major, then beta)
    float *wstart = pend + Q * C::PEND;        // WARPS x N states entering each warp chain
    float *ystart = wstart + WARPS * N;
    float *ring_all = ystart + N + 16;         // WARPS x STAGES x (padded matrix, vector)
    __shared__ int s_kind, s_seq, s_c, s_slot, s_abort, s_role;

    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const int g = lane >> 2, t = lane & 3;
    const int T = a.T;
    constexpr int S = C::STAGES;
    float *ring = ring_all + warp * S * C::STAGE_FLOATS;
    const int SW = w.sw, L = WARPS * SW;

    if (tid == 0) {
        s_abort = 0;
        s_role = (int)atomicAdd(&a.st->role_counter, 1u);
    }
    __syncthreads();
    if (s_role < w.resolvers) {
        if (warp < w.res_warps)
            resolver_big<N>(a, w, sm, s_role * w.res_warps + warp, w.resolvers * w.res_warps, lane);
        __syncthreads();
        if (tid == 0) scan_epilogue(a.st);
        return;
    }
    unsigned mb = 0;

    auto decode = [&](unsigned id, int &seq, int &c) {
        const unsigned j = id % (unsigned)w.Wd;
        const unsigned ws_ = id / (unsigned)w.Wd;
        seq = (int)(ws_ % (unsigned)a.B);
        const unsigned win = ws_ / (unsigned)a.B;
        c = (int)(win * (unsigned)w.Wd + j);
        if (c >= w.nch) c = -1;
    };
    int q_seq[Q], q_c[Q], q_head = 0, q_cnt = 0;
    bool exhausted = false;

    for (;;) {
        __syncthreads();
        if (tid == 0) {
            int kind = -1, seq = -1, c = -1, slot = 0;
            bool want_b = false;
            if (q_cnt > 0) {
                want_b = (q_cnt == Q) || exhausted;
                if (!want_b)
                    want_b = ld_relaxed_u64(w.starts + ((size_t)q_seq[q_head] * w.nch + q_c[q_head]) * N) != 0ull;
            }
            if (!want_b && !exhausted) {
                for (;;) {
                    const unsigned id = atomicAdd(&a.st->tile_counter, 1u);
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
        float *wagg = pend + s_slot * C::PEND;
        const int s0 = c * L;
        const int Lt = min(L, T - s0);
        const int p0 = warp * SW;
        const int cnt = min(SW, max(0, Lt - p0));
        const int sbase = s0 + p0;                             // scan position of the chain's first element
        const size_t tile_index = (size_t)seq * w.nch + c;
        const float *Jseq = a.J + (size_t)seq * T * NN;
        const float *bseq = a.b + (size_t)seq * T * N;
        // matrix of scan position s: forward J[s]; reverse J[T-s] (identity at s = 0); vector at t(s)
        auto mat_ptr = [&](int s) { return REV ? Jseq + (size_t)(T - s) * NN : Jseq + (size_t)s * NN; };
        auto pos_t = [&](int s) -> size_t { return REV ? (size_t)(T - 1 - s) : (size_t)s; };
        // chain position q -> ring stage q % S (one commit group per call, also past the end)
        auto issue = [&](int q) {
            const int s = sbase + q;
            const bool valid = q < cnt;
            issue_stage_n<N, REV>(ring + (q % S) * C::STAGE_FLOATS, valid ? mat_ptr(s) : nullptr,
                             valid ? bseq + pos_t(s) * N : nullptr, valid, REV && s == 0, lane);
        };

        if (kind == 0) {
            // ---------------------------------------------- A item
            float acc[MT][NT][4];
            identity_fragments<N>(acc, g, t);
            float yv[NT][2];
#pragma unroll
            for (int kk = 0; kk < NT; ++kk) { yv[kk][0] = 0.0f; yv[kk][1] = 0.0f; }
#pragma unroll
            for (int q = 0; q < S - 1; ++q) issue(q);
#pragma unroll 1
            for (int q = 0; q < cnt; ++q) {
                cp_async_wait_n<S - 2>();
                __syncwarp();                  // stage q landed for every lane; stage q-1 is free again
                issue(q + S - 1);
                const float *Ms = ring + (q % S) * C::STAGE_FLOATS;
                float jp[NT][NT][2], bg[NT], ynew[NT];
                load_pieces<N, REV>(jp, Ms, g, t);
#pragma unroll
                for (int nn = 0; nn < NT; ++nn) bg[nn] = Ms[N * RingRow<N, REV>::RS + 8 * nn + g];
                chain_step_n<N>(acc, jp);
                matvec_step<N>(yv, jp, bg, ynew, t);
            }
            cp_async_wait_n<0>();
            __syncwarp();
            store_aggregate<N>(warp + 1 < WARPS ? wagg + warp * AGG : ring, acc, yv, g, t);
            __syncthreads();
            if (warp == 0) {
                // tile aggregate = the same steps with the warp aggregates as positions (forward form)
                identity_fragments<N>(acc, g, t);
#pragma unroll
                for (int kk = 0; kk < NT; ++kk) { yv[kk][0] = 0.0f; yv[kk][1] = 0.0f; }
#pragma unroll 1
                for (int k = 0; k < WARPS; ++k) {
                    const float *ak = k + 1 < WARPS ? wagg + k * AGG : ring_all + (WARPS - 1) * S * C::STAGE_FLOATS;
                    float jp[NT][NT][2], bg[NT], ynew[NT];
                    load_pieces_smem<N>(jp, ak, g, t);
#pragma unroll
                    for (int nn = 0; nn < NT; ++nn) bg[nn] = ak[NN + 8 * nn + g];
                    chain_step_n<N>(acc, jp);
                    matvec_step<N>(yv, jp, bg, ynew, t);
                }
                store_aggregate<N>(w.aggs + tile_index * AGG, acc, yv, g, t);
                __threadfence();
                __syncwarp();
                if (lane == 0) st_release_u32(w.flags + tile_index, 1u);
            }
            continue;
        }

        // -------------------------------------------------- B item
#pragma unroll
        for (int q = 0; q < S - 1; ++q) issue(q);      // the chain's first positions fly while the state arrives
        if (warp == 1) {
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
        __syncthreads();
        if (s_abort) { cp_async_wait_n<0>(); break; }
        if (warp == 0) {
            // states entering each warp chain: walk the warp aggregates from the tile's entering state
            float yv[NT][2];
#pragma unroll
            for (int kk = 0; kk < NT; ++kk) { yv[kk][0] = ystart[8 * kk + 2 * t]; yv[kk][1] = ystart[8 * kk + 2 * t + 1]; }
#pragma unroll 1
            for (int k = 0; k < WARPS; ++k) {
                if (g == 0) {
#pragma unroll
                    for (int kk = 0; kk < NT; ++kk) {
                        wstart[k * N + 8 * kk + 2 * t] = yv[kk][0];
                        wstart[k * N + 8 * kk + 2 * t + 1] = yv[kk][1];
                    }
                }
                if (k + 1 == WARPS) break;
                const float *ak = wagg + k * AGG;
                float jp[NT][NT][2], bg[NT], ynew[NT];
                load_pieces_smem<N>(jp, ak, g, t);
#pragma unroll
                for (int nn = 0; nn < NT; ++nn) bg[nn] = ak[NN + 8 * nn + g];
                matvec_step<N>(yv, jp, bg, ynew, t);
            }
        }
        __syncthreads();
        {
            float yv[NT][2];
#pragma unroll
            for (int kk = 0; kk < NT; ++kk) {
                yv[kk][0] = wstart[warp * N + 8 * kk + 2 * t];
                yv[kk][1] = wstart[warp * N + 8 * kk + 2 * t + 1];
            }
#pragma unroll 1
            for (int q = 0; q < cnt; ++q) {
                const int s = sbase + q;
                cp_async_wait_n<S - 2>();
                __syncwarp();
                issue(q + S - 1);
                const float *Ms = ring + (q % S) * C::STAGE_FLOATS;
                float jp[NT][NT][2], bg[NT], ynew[NT];
                load_pieces<N, REV>(jp, Ms, g, t);
                const size_t vb = ((size_t)seq * T + pos_t(s)) * N;
#pragma unroll
                for (int nn = 0; nn < NT; ++nn) bg[nn] = Ms[N * RingRow<N, REV>::RS + 8 * nn + g];
                matvec_step<N>(yv, jp, bg, ynew, t);
                if (t == 0) {
#pragma unroll
                    for (int nn = 0; nn < NT; ++nn) {
                        if (a.yold) mb = max(mb, absdiff_bits(ynew[nn], __ldg(a.yold + vb + 8 * nn + g)));
                        a.y[vb + 8 * nn + g] = ynew[nn];
                    }
                }
            }
            cp_async_wait_n<0>();
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
