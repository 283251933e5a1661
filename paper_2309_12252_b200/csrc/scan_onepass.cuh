// Single-pass chunked scan of the linear recurrence for n in {1, 2, 4, 8}:
// J and b are read from HBM exactly once, y written once.
//
//   * A tile of L consecutive positions of one sequence is staged in shared
//     memory by bulk asynchronous copies (cp.async.bulk + mbarrier), one copy
//     per "chain run" so that runs can be padded by 16 bytes: with the pad the
//     run stride is an odd number of 16-byte units and the 128-bit shared
//     loads of the chains of a warp fall in distinct banks.
//   * A chain is LPC lanes that own S consecutive positions.  Each lane keeps
//     COLS = n / LPC columns of the running product A (and the whole vector
//     beta, redundantly) in registers and multiplies the next J_t, broadcast
//     from shared memory, onto them:  (A, beta) <- (J_t A, J_t beta + b_t).
//   * Chain aggregates are combined per warp and per tile in shared memory;
//     the tile aggregate is published to global memory and the state entering
//     the tile is obtained by a decoupled look-back over earlier tiles of the
//     same sequence.  Tile ids are handed out by an atomic counter, ordered so
//     that a tile only ever waits on lower ids (no co-residency assumption),
//     and every wait is bounded: on expiry the kernel raises FLAG_TIMEOUT and
//     all CTAs drain.
//   * The tile is then replayed from its entering state (matrix-vector work
//     only), y overwrites b in shared memory and is streamed out with
//     coalesced stores fused with the max |y - y_old| reduction.
//
// reverse scans (adjoint) use the same kernel with reversed run indexing and
// transposed register access.
#pragma once
#include "common.cuh"

namespace deer {

template <int N> struct OnePass {
    static constexpr int LPC = (N >= 4) ? 4 : N;       // lanes per chain
    static constexpr int COLS = N / LPC;               // columns of A per lane
    static constexpr int S = (N == 8) ? 6 : (N == 4) ? 24 : (N == 2) ? 40 : 64;   // positions per chain
    static constexpr int THREADS = 128;
    static constexpr int WARPS = THREADS / 32;
    static constexpr int CHAINS = THREADS / LPC;
    static constexpr int CPW = CHAINS / WARPS;         // chains per warp
    static constexpr int L = CHAINS * S;               // positions per tile
    static constexpr int JRUN = S * N * N + 4;         // floats per chain run of J, padded
    static constexpr int BRUN = S * N + 4;             // floats per chain run of b / y, padded
    static constexpr int AGG = N * N + N;              // floats of one aggregate (A row-major, then beta)
    static constexpr int SM_FLOATS = CHAINS * JRUN + CHAINS * BRUN + CHAINS * AGG + WARPS * AGG +
                                     WARPS * 2 * AGG + AGG + CHAINS * N + WARPS * N + N;
    static constexpr size_t SMEM = SM_FLOATS * sizeof(float) + 64;
    static_assert((JRUN / 4) % 2 == 1 && (BRUN / 4) % 2 == 1, "run strides must be odd in 16-byte units");
};

struct OnePassWs {
    unsigned *flags;     // [B*nch]   0 = nothing, 1 = aggregate published, 2 = inclusive state published
    float *aggs;         // [B*nch][n*n+n]
    float *incl;         // [B*nch][n]  state leaving the tile
    int nch, Wd, nwin;   // tiles per sequence, tiles per sequence per window, windows
    unsigned total_ids;
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
    if (lane < N) {
        float acc = agg[N * N + lane];
#pragma unroll
        for (int k = 0; k < N; ++k) acc = fmaf(agg[lane * N + k], in[k], acc);
        out[lane] = acc;
    }
    __syncwarp();
}

template <int N, bool REV>
__global__ void __launch_bounds__(OnePass<N>::THREADS) scan_onepass_kernel(ScanArgs a, OnePassWs w)
{
    using C = OnePass<N>;
    constexpr int LPC = C::LPC, COLS = C::COLS, S = C::S, CHAINS = C::CHAINS, CPW = C::CPW;
    constexpr int JRUN = C::JRUN, BRUN = C::BRUN, AGG = C::AGG, WARPS = C::WARPS, NN = N * N;

    extern __shared__ __align__(16) float smem[];
    float *sJ = smem;
    float *sB = sJ + CHAINS * JRUN;
    float *agg = sB + CHAINS * BRUN;
    float *wagg = agg + CHAINS * AGG;
    float *tmp = wagg + WARPS * AGG;
    float *tagg = tmp + WARPS * 2 * AGG;
    float *cstart = tagg + AGG;
    float *wstart = cstart + CHAINS * N;
    float *ystart = wstart + WARPS * N;
    uint64_t *bar = (uint64_t *)(((uintptr_t)(ystart + N) + 15) & ~(uintptr_t)15);
    __shared__ int s_seq, s_c, s_abort;

    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const int chain = tid / LPC, sub = tid % LPC;
    const unsigned chain_mask = (LPC == 32) ? 0xffffffffu : (((1u << LPC) - 1u) << (lane & ~(LPC - 1)));
    const int chain_lane0 = lane & ~(LPC - 1);
    const int T = a.T;

    if (tid == 0) { mbar_init(bar, 1); s_abort = 0; }
    fence_proxy_async();
    __syncthreads();
    unsigned phase = 0;
    unsigned mb = 0;          // running max |y - yold| bits of this thread

    for (;;) {
        __syncthreads();      // previous tile done with shared memory and with s_seq / s_c
        if (tid == 0) {
            int seq = -1, c = -1;
            for (;;) {
                unsigned id = atomicAdd(&a.st->tile_counter, 1u);
                if (id >= w.total_ids) break;
                // id = (window * B + seq) * Wd + j
                unsigned j = id % (unsigned)w.Wd;
                unsigned ws_ = id / (unsigned)w.Wd;
                unsigned sq = ws_ % (unsigned)a.B;
                unsigned win = ws_ / (unsigned)a.B;
                int cc = (int)(win * (unsigned)w.Wd + j);
                if (cc < w.nch) { seq = (int)sq; c = cc; break; }
            }
            s_seq = seq; s_c = c;
        }
        __syncthreads();
        if (s_c < 0 || s_abort) break;
        const int seq = s_seq, c = s_c;
        const int s0 = c * C::L;
        const int Lt = min(C::L, T - s0);
        const size_t tile_index = (size_t)seq * w.nch + c;

        // ------------------------------------------------ stage the tile (warp 0 issues, everybody waits)
        if (warp == 0) {
            fence_proxy_async();
            unsigned bytes = 0;
#pragma unroll 1
            for (int r = lane; r < CHAINS; r += 32) {
                int cnt = min(S, max(0, Lt - r * S));
                if (cnt <= 0) continue;
                size_t p_lo = REV ? (size_t)(T - (s0 + r * S + cnt)) : (size_t)(s0 + r * S);   // first t of the run
                int jcnt = cnt;
                size_t j_lo = p_lo;
                if (REV) { j_lo = p_lo + 1; if (s0 + r * S == 0) jcnt = cnt - 1; }
                const float *jsrc = a.J + ((size_t)seq * T + j_lo) * NN;
                const float *bsrc = a.b + ((size_t)seq * T + p_lo) * N;
                unsigned jb = (unsigned)jcnt * NN * 4u, bb = (unsigned)cnt * N * 4u;
                if (jb && ((uintptr_t)jsrc & 15) == 0 && (jb & 15) == 0) bytes += jb;
                if (((uintptr_t)bsrc & 15) == 0 && (bb & 15) == 0) bytes += bb;
            }
#pragma unroll
            for (int o = 16; o > 0; o >>= 1) bytes += __shfl_xor_sync(0xffffffffu, bytes, o);
            if (lane == 0) mbar_arrive_expect_tx(bar, bytes);
            __syncwarp();
#pragma unroll 1
            for (int r = lane; r < CHAINS; r += 32) {
                int cnt = min(S, max(0, Lt - r * S));
                if (cnt <= 0) continue;
                size_t p_lo = REV ? (size_t)(T - (s0 + r * S + cnt)) : (size_t)(s0 + r * S);
                int jcnt = cnt;
                size_t j_lo = p_lo;
                if (REV) { j_lo = p_lo + 1; if (s0 + r * S == 0) jcnt = cnt - 1; }
                const float *jsrc = a.J + ((size_t)seq * T + j_lo) * NN;
                const float *bsrc = a.b + ((size_t)seq * T + p_lo) * N;
                unsigned jb = (unsigned)jcnt * NN * 4u, bb = (unsigned)cnt * N * 4u;
                float *jd = sJ + r * JRUN, *bd = sB + r * BRUN;
                if (jb) {
                    if (((uintptr_t)jsrc & 15) == 0 && (jb & 15) == 0) bulk_g2s(jd, jsrc, jb, bar);
                    else for (int i = 0; i < jcnt * NN; ++i) jd[i] = __ldg(jsrc + i);
                }
                if (((uintptr_t)bsrc & 15) == 0 && (bb & 15) == 0) bulk_g2s(bd, bsrc, bb, bar);
                else for (int i = 0; i < cnt * N; ++i) bd[i] = __ldg(bsrc + i);
            }
        }
        {
            unsigned spins = 0;
            while (!mbar_try_wait(bar, phase)) {
                if (++spins > (SPIN_LIMIT >> 2)) { atomicOr(&a.st->flags, FLAG_TIMEOUT); s_abort = 1; break; }
            }
            phase ^= 1u;
        }
        __syncthreads();      // plain-copied runs visible; s_abort visible
        if (s_abort) break;

        // ------------------------------------------------ reduce: chain aggregate in registers
        const int cnt = min(S, max(0, Lt - chain * S));
        const float *cJ = sJ + chain * JRUN;
        float *cB = sB + chain * BRUN;
        float A[N][COLS], be[N];
#pragma unroll
        for (int i = 0; i < N; ++i) {
            be[i] = 0.0f;
#pragma unroll
            for (int cc = 0; cc < COLS; ++cc) A[i][cc] = (i == sub * COLS + cc) ? 1.0f : 0.0f;
        }
#pragma unroll 1
        for (int q = 0; q < cnt; ++q) {
            const int li = REV ? cnt - 1 - q : q;
            const bool ident = REV && (s0 + chain * S + q == 0);
            const float *Je = cJ + li * NN;
            const float *bv = cB + li * N;
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
                for (int i = 0; i < N; ++i) be[i] = bv[i];
                continue;
            }
            float Jr[NN];
            if constexpr (NN >= 4) {
#pragma unroll
                for (int v = 0; v < NN / 4; ++v) {
                    float4 f = reinterpret_cast<const float4 *>(Je)[v];
                    Jr[4 * v] = f.x; Jr[4 * v + 1] = f.y; Jr[4 * v + 2] = f.z; Jr[4 * v + 3] = f.w;
                }
            } else {
                Jr[0] = Je[0];
            }
            float An[N][COLS], bn[N];
#pragma unroll
            for (int i = 0; i < N; ++i) {
                bn[i] = bv[i];
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

        // ------------------------------------------------ warp aggregate, then tile aggregate (warp 0)
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
            // ---------------------------------------------- publish / look back
            unsigned *flags = w.flags + (size_t)seq * w.nch;
            const float *aggs = w.aggs + (size_t)seq * w.nch * AGG;
            const float *incl = w.incl + (size_t)seq * w.nch * N;
            bool ok = true;
            if (c > 0) {
                float *g = w.aggs + tile_index * AGG;
                for (int o = lane; o < AGG; o += 32) g[o] = tagg[o];
                __threadfence();
                __syncwarp();
                if (lane == 0) st_release_u32(flags + c, 1u);
                // nearest earlier tile with its inclusive state published; all tiles in between need aggregates
                int hi = c - 1, p = -2;
                unsigned spins = 0;
                while (p == -2) {
                    const int j = hi - lane;
                    const unsigned f = (j >= 0) ? ld_acquire_u32(flags + j) : 2u;
                    const unsigned m2 = __ballot_sync(0xffffffffu, f == 2u);
                    const unsigned m0 = __ballot_sync(0xffffffffu, f == 0u);
                    const int first2 = m2 ? (__ffs(m2) - 1) : 32;
                    const unsigned below = (first2 >= 32) ? 0xffffffffu : ((1u << first2) - 1u);
                    if (m0 & below) {
                        __nanosleep(64);
                        if (++spins > SPIN_LIMIT || ((spins & 1023u) == 0 &&
                                                     (*(volatile unsigned *)&a.st->flags & FLAG_TIMEOUT))) {
                            if (lane == 0) atomicOr(&a.st->flags, FLAG_TIMEOUT);
                            ok = false;
                            break;
                        }
                        continue;
                    }
                    if (first2 < 32) p = hi - first2;      // may be -1: the sequence start
                    else hi -= 32;
                }
                if (ok) {
                    __threadfence();
                    if (lane < N) ystart[lane] = (p < 0) ? (a.y0 ? a.y0[(size_t)seq * N + lane] : 0.0f)
                                                         : __ldcg(incl + (size_t)p * N + lane);
                    __syncwarp();
                    for (int j = p + 1; j < c; ++j) {
                        const float *g2 = aggs + (size_t)j * AGG;
                        float acc = 0.0f;
                        if (lane < N) {
                            acc = __ldcg(g2 + NN + lane);
#pragma unroll
                            for (int k = 0; k < N; ++k) acc = fmaf(__ldcg(g2 + lane * N + k), ystart[k], acc);
                        }
                        __syncwarp();
                        if (lane < N) ystart[lane] = acc;
                        __syncwarp();
                    }
                }
            } else {
                if (lane < N) ystart[lane] = a.y0 ? a.y0[(size_t)seq * N + lane] : 0.0f;
                __syncwarp();
            }
            if (ok) {
                // state leaving the tile -> inclusive flag, as early as possible
                if (lane < N) {
                    float acc = tagg[NN + lane];
#pragma unroll
                    for (int k = 0; k < N; ++k) acc = fmaf(tagg[lane * N + k], ystart[k], acc);
                    w.incl[tile_index * N + lane] = acc;
                }
                __threadfence();
                __syncwarp();
                if (lane == 0) st_release_u32(flags + c, 2u);
                // states entering each warp's first chain
                if (lane < N) wstart[lane] = ystart[lane];
                __syncwarp();
                for (int k = 0; k + 1 < WARPS; ++k)
                    matvec_smem<N>(wstart + (k + 1) * N, wagg + k * AGG, wstart + k * N, lane);
            } else if (lane == 0) {
                s_abort = 1;
            }
        }
        __syncthreads();
        if (s_abort) break;

        // ------------------------------------------------ states entering each chain (per warp)
        {
            float *cs = cstart + (warp * CPW) * N;
            if (lane < N) cs[lane] = wstart[warp * N + lane];
            __syncwarp();
            for (int k = 0; k + 1 < CPW; ++k)
                matvec_smem<N>(cs + (k + 1) * N, agg + (warp * CPW + k) * AGG, cs + k * N, lane);
        }

        // ------------------------------------------------ apply: replay the chain, y overwrites b
        {
            float y[N];
#pragma unroll
            for (int k = 0; k < N; ++k) y[k] = cstart[chain * N + k];
#pragma unroll 1
            for (int q = 0; q < cnt; ++q) {
                const int li = REV ? cnt - 1 - q : q;
                const bool ident = REV && (s0 + chain * S + q == 0);
                const float *Je = cJ + li * NN;
                float *bv = cB + li * N;
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
                                float4 f = reinterpret_cast<const float4 *>(Je + i * N)[v4];
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
            const size_t t_lo = REV ? (size_t)(T - s0 - Lt) : (size_t)s0;
            const size_t gbase = ((size_t)seq * T + t_lo) * N;
            float *yo = a.y + gbase;
            const float *yold = a.yold ? a.yold + gbase : nullptr;
            const int total = Lt * N;
            const bool vec = (!REV || N >= 4) && (((uintptr_t)yo & 15) == 0) && ((total & 3) == 0) &&
                             (!yold || ((uintptr_t)yold & 15) == 0);
            if (vec) {
                for (int g4 = tid; g4 < total / 4; g4 += C::THREADS) {
                    const int g = 4 * g4;
                    int off;
                    if (!REV) {
                        const int r = g / (S * N);
                        off = r * BRUN + (g - r * S * N);
                    } else {
                        const int e = g / N, i = g % N;
                        const int ps = Lt - 1 - e, r = ps / S, q = ps % S;
                        const int cr = min(S, Lt - r * S);
                        off = r * BRUN + (cr - 1 - q) * N + i;
                    }
                    float4 val = *reinterpret_cast<const float4 *>(sB + off);
                    if (yold) {
                        float4 o = __ldg(reinterpret_cast<const float4 *>(yold) + g4);
                        mb = max(mb, absdiff_bits(val.x, o.x)); mb = max(mb, absdiff_bits(val.y, o.y));
                        mb = max(mb, absdiff_bits(val.z, o.z)); mb = max(mb, absdiff_bits(val.w, o.w));
                    }
                    reinterpret_cast<float4 *>(yo)[g4] = val;
                }
            } else {
                for (int g = tid; g < total; g += C::THREADS) {
                    const int e = g / N, i = g % N;
                    int off;
                    if (!REV) {
                        const int r = e / S;
                        off = r * BRUN + (e - r * S) * N + i;
                    } else {
                        const int ps = Lt - 1 - e, r = ps / S, q = ps % S;
                        const int cr = min(S, Lt - r * S);
                        off = r * BRUN + (cr - 1 - q) * N + i;
                    }
                    float val = sB[off];
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
