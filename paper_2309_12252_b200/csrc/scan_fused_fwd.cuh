// The scan inside deer_gru_eval for n = 16 and n = 32 (J generated from coefficient rows), as two launches.
//
// The iteration runs in its Newton-update form (App. A.1: the same iteration as Eq. 3): the cell hands over
// the coefficient rows of J_t and the residual r_t = f_t - y_old,t, and the scan solves
//     d_t = J_t d_{t-1} + r_t,  d_{-1} = 0,          y_t = y_old,t + d_t,     err = max |y - y_old|
// (Eq. 9-10 for the update).  In this form the fixed point is f(y) = y whatever the accuracy of the linear
// solve, so every product below is a single TF32 MMA (operands truncated to 10 mantissa bits, fp32
// accumulate: relative error about 1e-3 in the update, which the next body removes).
//
//   * scan_fused_reduce_kernel -- the chunk reduce and the carries: persistent CTAs take tiles of WARPS chains
//     of SW positions; every warp folds its chain into (P, beta) as in scan_warpn_fused.cuh (J_t built from the
//     staged coefficient rows and W_h in shared memory, X <- X J_t^T on accumulator fragments, beta as an fp32
//     mat-vec chain); warp 0 combines the warp aggregates, writes the PREFIX aggregates of the tile (what maps the
//     state entering the tile to the state entering chain k) to global memory and publishes the tile aggregate;
//     resolver CTAs walk the tile aggregates of each sequence and write the state entering every tile.
//     Workers never wait: there are no replay items in this kernel.
//   * scan_fused_apply_kernel -- the replay of all chains, SIXTEEN chains per warp in lockstep on tensor cores.
//     With J_t = diag(k_r) W_hr + diag(a_z) W_hz + diag(k_n) W_hn + diag(z),
//         d_t = z . d + k_r . (W_hr d) + a_z . (W_hz d) + k_n . (W_hn d) + r_t        (d = d_{t-1})
//     and W_h is the same for every chain: the rows of the MMA A operand are the updates of 16 different chains,
//     the B operand is W_h^T, constant, in registers ([16, n] x [n, 3n] per step: 3 n^2 / 64 MMAs for 16
//     positions), and the coefficient rows enter elementwise in the epilogue.  J_t is never formed here.
//     Per step a warp stages 16 x (coefficient rows, r, y_old) into a warp-private cp.async ring (bulk copies of
//     128 ... 512 bytes, 48 per step, were measured several times slower).
#pragma once
#include <cuda_bf16.h>
#include "scan_warpn_fused.cuh"

namespace deer {

// d = a * b + c   (m16n8k16, A row-major 16x16, B 16x8, bf16 inputs, fp32 accumulate)
__device__ __forceinline__ void mma_bf16(float (&d)[4], const unsigned (&a)[4], const unsigned (&b)[2], const float (&c)[4])
{
    asm volatile("mma.sync.aligned.m16n8k16.row.col.f32.bf16.bf16.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%10,%11,%12,%13};"
                 : "=f"(d[0]), "=f"(d[1]), "=f"(d[2]), "=f"(d[3])
                 : "r"(a[0]), "r"(a[1]), "r"(a[2]), "r"(a[3]), "r"(b[0]), "r"(b[1]),
                   "f"(c[0]), "f"(c[1]), "f"(c[2]), "f"(c[3]));
}

// two floats rounded to nearest bf16, `lo` in the low half
__device__ __forceinline__ unsigned pack_bf16(float lo, float hi)
{
    const __nv_bfloat162 v = __floats2bfloat162_rn(lo, hi);
    return *reinterpret_cast<const unsigned *>(&v);
}

// packed bf16 arithmetic on register pairs (two values per 32-bit register, one instruction)
__device__ __forceinline__ unsigned hfma2_bf16(unsigned a, unsigned b, unsigned c)
{
    unsigned d;
    asm("fma.rn.bf16x2 %0, %1, %2, %3;" : "=r"(d) : "r"(a), "r"(b), "r"(c));
    return d;
}
__device__ __forceinline__ unsigned hmul2_bf16(unsigned a, unsigned b)
{
    unsigned d;
    asm("mul.rn.bf16x2 %0, %1, %2;" : "=r"(d) : "r"(a), "r"(b));
    return d;
}
__device__ __forceinline__ unsigned hadd2_bf16(unsigned a, unsigned b)
{
    unsigned d;
    asm("add.rn.bf16x2 %0, %1, %2;" : "=r"(d) : "r"(a), "r"(b));
    return d;
}

#ifndef DEER_FUSED_BF16
#define DEER_FUSED_BF16 1
#endif

template <int N> struct FusedFwd {
    using F = WarpNF<N, false>;
    static constexpr int NN = N * N, AGG = N * N + N, NT = N / 8, MT = N / 16;
    static constexpr int WARPS = F::WARPS, THREADS = F::THREADS;       // chains per tile of the reduce kernel
    static constexpr int CTAS_PER_SM = F::CTAS_PER_SM;                 // (sets the tile length: tiles per resident CTA)
    static constexpr bool BF16 = DEER_FUSED_BF16;                      // chain products of the reduce kernel as bf16 m16n8k16
    static constexpr int R_CTAS = 3;                                   // reduce kernel: CTAs per SM (n = 32: 168 registers, the weights as bf16 pairs)
    static constexpr int STAGES = F::STAGES, STAGE_FLOATS = F::STAGE_FLOATS, WS = F::WS;
    static constexpr int RES_WARPS = F::RES_WARPS, MAX_SEQ_PER_WARP = F::MAX_SEQ_PER_WARP;
    static constexpr int SM_WORK = WARPS * AGG + 16 + WARPS * STAGES * STAGE_FLOATS;
    static constexpr int SM_RES = F::SM_RES;
    static constexpr int SM_FLOATS = SM_WORK > SM_RES ? SM_WORK : SM_RES;
    static constexpr size_t SMEM = SM_FLOATS * sizeof(float) + 128;
    // apply kernel
    static constexpr int ROWS = 16;                    // chains per warp
    static constexpr int A_WARPS = 3, A_THREADS = 96, A_STAGES = 2;   // two CTAs per SM at n = 32: six warps, each one step ahead of itself
    static constexpr int ROW_FLOATS = 6 * N + 4;       // coefficient rows [N][4], r [N], y_old [N]; the pad keeps the
                                                       // 128-bit coefficient reads of a quarter-warp in distinct banks
    static constexpr int STAGE_A = ROWS * ROW_FLOATS;
    static constexpr size_t A_SMEM = sizeof(float) * (A_WARPS * A_STAGES * STAGE_A + A_WARPS * ROWS * N) + 128;
};

template <int N>
__global__ void __launch_bounds__(FusedFwd<N>::THREADS, FusedFwd<N>::R_CTAS) scan_fused_reduce_kernel(ScanArgs a, OnePassWs w)
{
    using C = FusedFwd<N>;
    constexpr int NN = C::NN, AGG = C::AGG, NT = C::NT, MT = C::MT, WARPS = C::WARPS, S = C::STAGES;
    pdl_prologue();
    if (loop_ended(a.st)) return;

    extern __shared__ __align__(16) float smem_raw[];
    float *sm = (float *)(((uintptr_t)smem_raw + 127) & ~(uintptr_t)127);
    float *wagg = sm;                          // WARPS warp aggregates (A row-major, then beta)
    float *ring_all = wagg + WARPS * AGG + 16; // WARPS x STAGES x (coefficients [N][4], vector [N])
    __shared__ int s_seq, s_c, s_role;

    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const int g = lane >> 2, t = lane & 3;
    const int T = a.T;
    float *ring = ring_all + warp * S * C::STAGE_FLOATS;
    const int SW = w.sw, L = WARPS * SW;
    // This lane's share of W_h stays in registers for the whole launch: the pieces it multiplies into its operand
    // pieces of J_t, {W[8nn+g][8kk+2t], W[8nn+g][8kk+2t+1]} per gate (3 n^2 / 32 values).  Read from shared memory
    // instead (12 KB per warp and position at n = 32) they kept the shared-memory pipe 69 % busy and bound the kernel.
    // (bf16 products: the pieces are kept as bf16 pairs, half the registers)
    float2 wR[C::BF16 ? 1 : NT][C::BF16 ? 1 : NT], wZ[C::BF16 ? 1 : NT][C::BF16 ? 1 : NT], wN[C::BF16 ? 1 : NT][C::BF16 ? 1 : NT];
    unsigned wRb[NT][NT], wZb[NT][NT], wNb[NT][NT];
#pragma unroll
    for (int nn = 0; nn < NT; ++nn)
#pragma unroll
        for (int kk = 0; kk < NT; ++kk) {
            const float *wp = a.Wh + (size_t)(8 * nn + g) * N + 8 * kk + 2 * t;
            const float2 r2 = __ldg(reinterpret_cast<const float2 *>(wp));
            const float2 z2 = __ldg(reinterpret_cast<const float2 *>(wp + NN));
            const float2 n2 = __ldg(reinterpret_cast<const float2 *>(wp + 2 * NN));
            if constexpr (C::BF16) {
                wRb[nn][kk] = pack_bf16(r2.x, r2.y); wZb[nn][kk] = pack_bf16(z2.x, z2.y); wNb[nn][kk] = pack_bf16(n2.x, n2.y);
            } else {
                wR[nn][kk] = r2; wZ[nn][kk] = z2; wN[nn][kk] = n2;
                wRb[nn][kk] = 0u; wZb[nn][kk] = 0u; wNb[nn][kk] = 0u;
            }
        }
    const bool d0 = g == 2 * t, d1 = g == 2 * t + 1;      // this lane's pieces touch the diagonal where nn == kk

    if (tid == 0) s_role = (int)atomicAdd(&a.st->role_counter, 1u);
    __syncthreads();
    if (s_role < w.resolvers) {
        if (warp < w.res_warps)
            resolver_big<N>(a, w, sm, s_role * w.res_warps + warp, w.resolvers * w.res_warps, lane);
        __syncthreads();
        if (tid == 0) scan_epilogue(a.st, false);
        return;
    }

    auto decode = [&](unsigned id, int &seq, int &c) {
        const unsigned j = id % (unsigned)w.Wd;
        const unsigned ws_ = id / (unsigned)w.Wd;
        seq = (int)(ws_ % (unsigned)a.B);
        const unsigned win = ws_ / (unsigned)a.B;
        c = (int)(win * (unsigned)w.Wd + j);
        if (c >= w.nch) c = -1;
    };
    // thread 0 claims tile ids one tile ahead: the atomic's round trip overlaps the current tile
    unsigned next_id = 0;
    if (tid == 0) next_id = atomicAdd(&a.st->tile_counter, 1u);

    for (;;) {
        __syncthreads();                       // the previous tile's combine is done with wagg and s_*
        if (tid == 0) {
            int seq = -1, c = -1;
            unsigned id = next_id;
            for (;;) {
                if (id >= w.total_ids) { c = -1; break; }
                decode(id, seq, c);
                if (c >= 0) break;
                id = atomicAdd(&a.st->tile_counter, 1u);
            }
            s_seq = seq; s_c = c;
            if (c >= 0) next_id = atomicAdd(&a.st->tile_counter, 1u);
        }
        __syncthreads();
        if (s_c < 0) break;
        const int seq = s_seq, c = s_c;
        const int s0 = c * L;
        const int Lt = min(L, T - s0);
        const int p0 = warp * SW;
        const int cnt = min(SW, max(0, Lt - p0));
        const int sbase = s0 + p0;
        const size_t tile_index = (size_t)seq * w.nch + c;
        const float *Cseq = a.J + (size_t)seq * T * 4 * N;      // coefficient rows {k_r, a_z, k_n, z}[N] per position
        const float *bseq = a.b + (size_t)seq * T * N;
        auto issue = [&](int q) {
            if (q < cnt) {
                float *dst = ring + (q % S) * C::STAGE_FLOATS;
                const float *cs = Cseq + (size_t)(sbase + q) * 4 * N, *bs = bseq + (size_t)(sbase + q) * N;
#pragma unroll
                for (int u = 0; u < (5 * N / 4 + 31) / 32; ++u) {
                    const int j = lane + 32 * u;
                    if (j < N) cp_async16(dst + 4 * j, cs + 4 * j);
                    else if (j < N + N / 4) cp_async16(dst + 4 * j, bs + 4 * (j - N));
                }
            }
            cp_async_commit();
        };

        float acc[MT][NT][4];
        identity_fragments<N>(acc, g, t);
        float yv[NT][2];
        float bacc[NT][2];                 // (bf16 form) beta, columns 8nn+2t, 8nn+2t+1, live in the lanes g == 0
#pragma unroll
        for (int kk = 0; kk < NT; ++kk) { yv[kk][0] = 0.0f; yv[kk][1] = 0.0f; bacc[kk][0] = 0.0f; bacc[kk][1] = 0.0f; }
#pragma unroll
        for (int q = 0; q < S - 1; ++q) issue(q);
#pragma unroll 1
        for (int q = 0; q < cnt; ++q) {
            cp_async_wait_n<S - 2>();
            __syncwarp();                  // stage q landed for every lane; stage q-1 is free again
            issue(q + S - 1);
            const float *Ms = ring + (q % S) * C::STAGE_FLOATS;
            // contraction block kk at a time: build the lane's pieces J_t[8nn+g][8kk+2t..+1] of every column block nn
            // from the coefficient rows and the weights in registers, multiply them into the new X (MT * NT
            // independent accumulators in flight) and into beta's partial sums
            float nacc[MT][NT][4];
            float nb[NT][4];               // (bf16 form) the beta row tile's new accumulators
            float4 cf[NT];
            float2 p2[NT];
#pragma unroll
            for (int nn = 0; nn < NT; ++nn) {
                cf[nn] = *reinterpret_cast<const float4 *>(Ms + 4 * (8 * nn + g));
                p2[nn] = make_float2(0.0f, 0.0f);
#pragma unroll
                for (int mm = 0; mm < MT; ++mm) { nacc[mm][nn][0] = 0.0f; nacc[mm][nn][1] = 0.0f; nacc[mm][nn][2] = 0.0f; nacc[mm][nn][3] = 0.0f; }
            }
            if constexpr (C::BF16) {
                // bf16 m16n8k16 products (half the MMAs of the TF32 form and chains half as long).  J_t is BUILT in packed
                // bf16 arithmetic, three instructions per pair of entries, and the result is the B fragment as it stands;
                // beta rides along as row 32 of X (a third row tile whose only live row is held by the lanes g == 0), so
                // its update is one more MMA per block instead of an fp32 mat-vec with its shuffles.  The accumulator
                // tiles 2j, 2j+1 of X are the A operand of contraction block j as they stand.
                unsigned cr[NT], cz[NT], cn[NT], zd[NT];
#pragma unroll
                for (int nn = 0; nn < NT; ++nn) {
                    cr[nn] = pack_bf16(cf[nn].x, cf[nn].x);
                    cz[nn] = pack_bf16(cf[nn].y, cf[nn].y);
                    cn[nn] = pack_bf16(cf[nn].z, cf[nn].z);
                    zd[nn] = pack_bf16(d0 ? cf[nn].w : 0.0f, d1 ? cf[nn].w : 0.0f);
                    nb[nn][0] = 0.0f; nb[nn][1] = 0.0f; nb[nn][2] = 0.0f; nb[nn][3] = 0.0f;
                }
                // all B fragments first: they do not depend on X, so their (three-deep) chains run while the previous
                // position's MMAs drain; written level by level so that independent instructions follow one another
                unsigned bf[NT / 2][NT][2];
#pragma unroll
                for (int j = 0; j < NT / 2; ++j)
#pragma unroll
                    for (int nn = 0; nn < NT; ++nn)
#pragma unroll
                        for (int h = 0; h < 2; ++h) bf[j][nn][h] = hmul2_bf16(cn[nn], wNb[nn][2 * j + h]);
#pragma unroll
                for (int j = 0; j < NT / 2; ++j)
#pragma unroll
                    for (int nn = 0; nn < NT; ++nn)
#pragma unroll
                        for (int h = 0; h < 2; ++h) bf[j][nn][h] = hfma2_bf16(cz[nn], wZb[nn][2 * j + h], bf[j][nn][h]);
#pragma unroll
                for (int j = 0; j < NT / 2; ++j)
#pragma unroll
                    for (int nn = 0; nn < NT; ++nn)
#pragma unroll
                        for (int h = 0; h < 2; ++h) {
                            bf[j][nn][h] = hfma2_bf16(cr[nn], wRb[nn][2 * j + h], bf[j][nn][h]);
                            if (nn == 2 * j + h) bf[j][nn][h] = hadd2_bf16(bf[j][nn][h], zd[nn]);
                        }
                unsigned af[NT / 2][MT + 1][4];
#pragma unroll
                for (int j = 0; j < NT / 2; ++j) {
#pragma unroll
                    for (int mm = 0; mm < MT; ++mm) {
                        af[j][mm][0] = pack_bf16(acc[mm][2 * j][0], acc[mm][2 * j][1]);
                        af[j][mm][1] = pack_bf16(acc[mm][2 * j][2], acc[mm][2 * j][3]);
                        af[j][mm][2] = pack_bf16(acc[mm][2 * j + 1][0], acc[mm][2 * j + 1][1]);
                        af[j][mm][3] = pack_bf16(acc[mm][2 * j + 1][2], acc[mm][2 * j + 1][3]);
                    }
                    af[j][MT][0] = pack_bf16(bacc[2 * j][0], bacc[2 * j][1]);
                    af[j][MT][1] = 0u;
                    af[j][MT][2] = pack_bf16(bacc[2 * j + 1][0], bacc[2 * j + 1][1]);
                    af[j][MT][3] = 0u;
                }
#pragma unroll
                for (int j = 0; j < NT / 2; ++j)
#pragma unroll
                    for (int nn = 0; nn < NT; ++nn) {
#pragma unroll
                        for (int mm = 0; mm < MT; ++mm) mma_bf16(nacc[mm][nn], af[j][mm], bf[j][nn], nacc[mm][nn]);
                        mma_bf16(nb[nn], af[j][MT], bf[j][nn], nb[nn]);
                    }
            } else {
#pragma unroll
            for (int kk = 0; kk < NT; ++kk) {
                unsigned af[MT][4];
#pragma unroll
                for (int mm = 0; mm < MT; ++mm) {
                    af[mm][0] = __float_as_uint(acc[mm][kk][0]); af[mm][1] = __float_as_uint(acc[mm][kk][2]);
                    af[mm][2] = __float_as_uint(acc[mm][kk][1]); af[mm][3] = __float_as_uint(acc[mm][kk][3]);
                }
                const float2 ypair = make_float2(yv[kk][0], yv[kk][1]);
#pragma unroll
                for (int nn = 0; nn < NT; ++nn) {
                    const float2 cx = make_float2(cf[nn].x, cf[nn].x), cy = make_float2(cf[nn].y, cf[nn].y),
                                 cz = make_float2(cf[nn].z, cf[nn].z);
                    float2 v = ffma2(cx, wR[nn][kk], ffma2(cy, wZ[nn][kk], fmul2(cz, wN[nn][kk])));
                    if (nn == kk) { v.x += d0 ? cf[nn].w : 0.0f; v.y += d1 ? cf[nn].w : 0.0f; }
                    const unsigned bf[2] = {__float_as_uint(v.x), __float_as_uint(v.y)};
#pragma unroll
                    for (int mm = 0; mm < MT; ++mm) mma_tf32(nacc[mm][nn], af[mm], bf, nacc[mm][nn]);
                    p2[nn] = ffma2(v, ypair, p2[nn]);
                }
            }
            }
#pragma unroll
            for (int mm = 0; mm < MT; ++mm)
#pragma unroll
                for (int nn = 0; nn < NT; ++nn)
#pragma unroll
                    for (int i = 0; i < 4; ++i) acc[mm][nn][i] = nacc[mm][nn][i];
            if constexpr (C::BF16) {
                // beta <- beta J_t^T + r_t: the live row of the tile, columns 8nn+2t, 8nn+2t+1 in the lanes g == 0
#pragma unroll
                for (int nn = 0; nn < NT; ++nn) {
                    float2 r2 = make_float2(0.0f, 0.0f);
                    if (g == 0) r2 = *reinterpret_cast<const float2 *>(Ms + 4 * N + 8 * nn + 2 * t);
                    bacc[nn][0] = nb[nn][0] + r2.x;
                    bacc[nn][1] = nb[nn][1] + r2.y;
                }
            } else {
                float ynew[NT];
#pragma unroll
                for (int nn = 0; nn < NT; ++nn) {
                    float part = p2[nn].x + p2[nn].y;
                    part += __shfl_xor_sync(0xffffffffu, part, 1);
                    part += __shfl_xor_sync(0xffffffffu, part, 2);
                    ynew[nn] = part + Ms[4 * N + 8 * nn + g];
                }
#pragma unroll
                for (int kk = 0; kk < NT; ++kk) {
                    yv[kk][0] = __shfl_sync(0xffffffffu, ynew[kk], 4 * (2 * t));
                    yv[kk][1] = __shfl_sync(0xffffffffu, ynew[kk], 4 * (2 * t + 1));
                }
            }
        }
        cp_async_wait_n<0>();
        __syncwarp();
        if constexpr (C::BF16) {
            // beta from the lanes g == 0 to every lane's (2t, 2t+1) pairs, as store_aggregate takes it
#pragma unroll
            for (int kk = 0; kk < NT; ++kk) {
                yv[kk][0] = __shfl_sync(0xffffffffu, bacc[kk][0], t);
                yv[kk][1] = __shfl_sync(0xffffffffu, bacc[kk][1], t);
            }
        }
        store_aggregate<N>(wagg + warp * AGG, acc, yv, g, t);
        __syncthreads();
        if (warp == 0) {
            // prefix aggregates of the tile: the same steps with the warp aggregates as positions
            identity_fragments<N>(acc, g, t);
#pragma unroll
            for (int kk = 0; kk < NT; ++kk) { yv[kk][0] = 0.0f; yv[kk][1] = 0.0f; }
#pragma unroll 1
            for (int k = 0; k < WARPS; ++k) {
                const float *ak = wagg + k * AGG;
                float jp[NT][NT][2], bg[NT], ynew[NT];
                load_pieces_smem<N>(jp, ak, g, t);
#pragma unroll
                for (int nn = 0; nn < NT; ++nn) bg[nn] = ak[NN + 8 * nn + g];
                chain_step_n1<N>(acc, jp);
                matvec_step<N>(yv, jp, bg, ynew, t);
                float *dst = k + 1 < WARPS ? w.pfx + (tile_index * (WARPS - 1) + k) * AGG : w.aggs + tile_index * AGG;
                store_aggregate<N>(dst, acc, yv, g, t);
            }
            __threadfence();
            __syncwarp();
            if (lane == 0) st_release_u32(w.flags + tile_index, 1u);
        }
    }
    __syncthreads();
    if (tid == 0) scan_epilogue(a.st, false);
}

template <int N>
__global__ void __launch_bounds__(FusedFwd<N>::A_THREADS) scan_fused_apply_kernel(ScanArgs a, OnePassWs w)
{
    static_assert(N == 16 || N == 32, "n = 64 has a replay kernel of its own (scan_fused_fwd64.cuh)");
    using C = FusedFwd<N>;
    constexpr int NN = C::NN, AGG = C::AGG, NT = C::NT, ROWS = C::ROWS, RF = C::ROW_FLOATS, S = C::A_STAGES;
    constexpr int WA = C::WARPS;                       // chains per tile of the reduce kernel
    pdl_prologue();
    if (loop_ended(a.st)) return;

    extern __shared__ __align__(16) float smem_raw[];
    float *sm = (float *)(((uintptr_t)smem_raw + 127) & ~(uintptr_t)127);
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const int g = lane >> 2, t = lane & 3;
    float *ring = sm + warp * S * C::STAGE_A;
    float *yin = sm + C::A_WARPS * S * C::STAGE_A + warp * ROWS * N;

    // B operand of every step: W_h^T, contraction index renamed so that an accumulator fragment is the next A operand
    unsigned wf[NT][3 * NT][2];
#pragma unroll
    for (int kk = 0; kk < NT; ++kk)
#pragma unroll
        for (int nn = 0; nn < 3 * NT; ++nn) {
            const float2 v = __ldg(reinterpret_cast<const float2 *>(a.Wh + (size_t)(8 * nn + g) * N + 8 * kk + 2 * t));
            wf[kk][nn][0] = __float_as_uint(v.x); wf[kk][nn][1] = __float_as_uint(v.y);
        }

    const int T = a.T, SW = w.sw;
    const long long nchain = (T + SW - 1) / SW;
    const long long total = (long long)a.B * nchain;
    const long long groups = (total + ROWS - 1) / ROWS;
    unsigned mb = 0;
    unsigned it0 = 0;                                  // ring steps consumed so far (the stage of the next one)

    for (long long grp = (long long)blockIdx.x * C::A_WARPS + warp; grp < groups; grp += (long long)gridDim.x * C::A_WARPS) {
        // geometry of this lane's row (lanes l and l + 16 describe row l)
        const int row = lane & 15;
        const long long gid = grp * ROWS + row;
        const bool rv = gid < total;
        const long long seq = rv ? gid / nchain : 0;
        const int q = rv ? (int)(gid - seq * nchain) : 0;
        const int len = rv ? min(SW, T - q * SW) : 0;
        const size_t e0 = (size_t)seq * T + (size_t)q * SW;          // first position of the row's chain
        const size_t tile_index = (size_t)seq * w.nch + q / WA;
        const int kin = q % WA;
        int maxlen = len;
#pragma unroll
        for (int o = 8; o > 0; o >>= 1) maxlen = max(maxlen, __shfl_xor_sync(0xffffffffu, maxlen, o));

        // ---- updates entering the 16 chains: the tile's entering update through the tile's prefix aggregate
        for (int r = 0; r < ROWS; ++r) {
            const int vr = __shfl_sync(0xffffffffu, (int)rv, r);
            const unsigned long long tix = __shfl_sync(0xffffffffu, (unsigned long long)tile_index, r);
            const int kr = __shfl_sync(0xffffffffu, kin, r);
            {
                float val = 0.0f;
                if (vr) {
                    float yl = 0.0f;
                    if (lane < N) yl = __uint_as_float((unsigned)(ld_relaxed_u64(w.starts + tix * N + lane) & 0xffffffffull));
                    val = yl;
                    if (kr > 0) {
                        const float *ag = w.pfx + (tix * (WA - 1) + (kr - 1)) * AGG;
                        const float *arow = ag + (size_t)(lane < N ? lane : 0) * N;
                        float acc0 = (lane < N) ? __ldcg(ag + NN + lane) : 0.0f;
#pragma unroll
                        for (int j4 = 0; j4 < N / 4; ++j4) {
                            const float4 av = __ldcg(reinterpret_cast<const float4 *>(arow) + j4);
                            acc0 = fmaf(av.x, __shfl_sync(0xffffffffu, yl, (4 * j4) & 31), acc0);
                            acc0 = fmaf(av.y, __shfl_sync(0xffffffffu, yl, (4 * j4 + 1) & 31), acc0);
                            acc0 = fmaf(av.z, __shfl_sync(0xffffffffu, yl, (4 * j4 + 2) & 31), acc0);
                            acc0 = fmaf(av.w, __shfl_sync(0xffffffffu, yl, (4 * j4 + 3) & 31), acc0);
                        }
                        val = acc0;
                    }
                }
                if (lane < N) yin[r * N + lane] = val;
            }
        }
        __syncwarp();
        float d[NT][4];
#pragma unroll
        for (int nn = 0; nn < NT; ++nn) {
            const float2 lo = *reinterpret_cast<const float2 *>(yin + g * N + 8 * nn + 2 * t);
            const float2 hi = *reinterpret_cast<const float2 *>(yin + (g + 8) * N + 8 * nn + 2 * t);
            d[nn][0] = lo.x; d[nn][1] = lo.y; d[nn][2] = hi.x; d[nn][3] = hi.y;
        }
        __syncwarp();
        // rows g and g + 8 of this lane's fragments
        const int len_lo = __shfl_sync(0xffffffffu, len, g), len_hi = __shfl_sync(0xffffffffu, len, g + 8);
        const unsigned long long e_lo = __shfl_sync(0xffffffffu, (unsigned long long)e0, g);
        const unsigned long long e_hi = __shfl_sync(0xffffffffu, (unsigned long long)e0, g + 8);
        float *yp[2] = {a.y + e_lo * N + 2 * t, a.y + e_hi * N + 2 * t};
        const int lens[2] = {len_lo, len_hi};

        // one step into ring stage (it0 + s) % S (always one commit group).  Eight lanes copy 128 contiguous bytes of a
        // row, so a warp instruction covers four rows with one full line each: lane l serves the rows 4k + (l >> 3),
        // k = 0 .. 3, whose chain starts and lengths it fetches from the lanes that own them
        const int rsub = lane >> 3, cpos = 4 * (lane & 7);
        unsigned long long e0q[4];
        int lenq[4];
#pragma unroll
        for (int k = 0; k < 4; ++k) {
            e0q[k] = __shfl_sync(0xffffffffu, (unsigned long long)e0, 4 * k + rsub);
            lenq[k] = __shfl_sync(0xffffffffu, len, 4 * k + rsub);
        }
        auto issue = [&](int s) {
            float *stg_dst = ring + ((it0 + (unsigned)s) % S) * C::STAGE_A + rsub * RF + cpos;
#pragma unroll
            for (int k = 0; k < 4; ++k) {
                if (s < lenq[k]) {
                    float *dst = stg_dst + 4 * k * RF;
                    const size_t e = (size_t)e0q[k] + (size_t)s;
                    const float *sc = a.J + e * 4 * N + cpos, *sr = a.b + e * N + cpos, *so = a.yold + e * N + cpos;
#pragma unroll
                    for (int j = 0; j < N / 8; ++j) cp_async16(dst + 32 * j, sc + 32 * j);
#pragma unroll
                    for (int j = 0; j < (N + 31) / 32; ++j) {
                        if (N >= 32 || cpos < N) {
                            cp_async16(dst + 4 * N + 32 * j, sr + 32 * j);
                            cp_async16(dst + 5 * N + 32 * j, so + 32 * j);
                        }
                    }
                }
            }
            cp_async_commit();
        };
#pragma unroll
        for (int s = 0; s < S - 1; ++s) issue(s);

#pragma unroll 1
        for (int s = 0; s < maxlen; ++s) {
            cp_async_wait_n<S - 2>();
            __syncwarp();                      // step s landed for every lane; the stage of step s - 1 is free again
            issue(s + S - 1);
            const unsigned stg = (it0 + (unsigned)s) % S;
            // U = D W_h^T : [16 chains, n] x [n, 3n]
            float U[3 * NT][4];
#pragma unroll
            for (int nn = 0; nn < 3 * NT; ++nn) { U[nn][0] = 0.0f; U[nn][1] = 0.0f; U[nn][2] = 0.0f; U[nn][3] = 0.0f; }
#pragma unroll
            for (int kk = 0; kk < NT; ++kk) {
                const unsigned af[4] = {__float_as_uint(d[kk][0]), __float_as_uint(d[kk][2]), __float_as_uint(d[kk][1]),
                                        __float_as_uint(d[kk][3])};
#pragma unroll
                for (int nn = 0; nn < 3 * NT; ++nn) mma_tf32(U[nn], af, wf[kk][nn], U[nn]);
            }
            const float *st = ring + stg * C::STAGE_A;
#pragma unroll
            for (int h = 0; h < 2; ++h) {
                if (s < lens[h]) {
                    const float *rs = st + (g + 8 * h) * RF;
#pragma unroll
                    for (int nn = 0; nn < NT; ++nn) {
                        const int col = 8 * nn + 2 * t;
                        const float4 c0 = *reinterpret_cast<const float4 *>(rs + 4 * col);
                        const float4 c1 = *reinterpret_cast<const float4 *>(rs + 4 * col + 4);
                        const float2 r2 = *reinterpret_cast<const float2 *>(rs + 4 * N + col);
                        const float2 yo = *reinterpret_cast<const float2 *>(rs + 5 * N + col);
                        float dx = fmaf(c0.w, d[nn][2 * h], r2.x), dy = fmaf(c1.w, d[nn][2 * h + 1], r2.y);
                        dx = fmaf(c0.x, U[nn][2 * h], dx);              dy = fmaf(c1.x, U[nn][2 * h + 1], dy);
                        dx = fmaf(c0.y, U[NT + nn][2 * h], dx);         dy = fmaf(c1.y, U[NT + nn][2 * h + 1], dy);
                        dx = fmaf(c0.z, U[2 * NT + nn][2 * h], dx);     dy = fmaf(c1.z, U[2 * NT + nn][2 * h + 1], dy);
                        d[nn][2 * h] = dx; d[nn][2 * h + 1] = dy;
                        const float2 yn = make_float2(yo.x + dx, yo.y + dy);
                        mb = max(mb, absdiff_bits(yn.x, yo.x));
                        mb = max(mb, absdiff_bits(yn.y, yo.y));
                        *reinterpret_cast<float2 *>(yp[h] + (size_t)s * N + 8 * nn) = yn;
                    }
                }
            }
        }
        cp_async_wait_n<0>();
        __syncwarp();
        it0 += (unsigned)maxlen;
    }
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) mb = max(mb, __shfl_xor_sync(0xffffffffu, mb, o));
    if (lane == 0 && mb) { atomicMax(&a.st->err_bits, mb); __threadfence(); }
    __syncthreads();
    if (tid == 0) scan_epilogue(a.st, true);
}

}  // namespace deer
