// Single-pass scans for n = 16 and n = 32 inside deer_gru_eval and deer_gru_vjp, with J_t generated on the fly.
//
// The GRU Jacobian at a position is a function of four n-vectors and the shared hidden weights,
//     J = diag(k_r) W_hr + diag(a_z) W_hz + diag(k_n) W_hn + diag(z)
// (k_r = a_n q r (1-r), k_n = a_n r, a_z = (h - c) z (1-z), a_n = (1-z)(1-c^2); Sec. 3.1 / Eq. 5 with the
// closed-form GRU derivative), so the cell writes 16 n bytes per position instead of 4 n^2 and this
// kernel, identical to scan_warpn_kernel in everything else (both directions), builds the lane's
// operand pieces of J_t (forward) or J_{t+1}^T (reverse; identity at the first scan position: coefficient
// rows {0,0,0,1}) from the staged coefficient rows and W_h kept in shared memory: 3 n^2 FMAs per
// position and visit on the fp32 pipes in exchange for n/5 times less memory traffic.
//
// The forward kernel (inside deer_gru_eval) runs the iteration in its Newton-update form (App. A.1, shown there
// to be the same iteration as Eq. 3): the cell hands over the residual f - y_old, the scan solves
// d_t = J_t d_{t-1} + (f - y_old)_t from d_{-1} = 0 and writes y = y_old + d, err = max|d|.  In this form the
// fixed point is f(y) = y whatever the accuracy of the linear solve, so the chain products of the A item are
// single TF32 MMAs (no hi/lo split: a third of the tensor work and none of the split instructions); the
// replay of the B item stays fp32.  The reverse kernel (the gradient's one-shot solve) keeps 3 x TF32.
#pragma once
#include "scan_warpn.cuh"

namespace deer {

template <int N, bool REV = false> struct WarpNF {
    using B_ = WarpN<N>;
    static constexpr int NN = N * N, AGG = N * N + N, NT = N / 8, MT = N / 16;
    static constexpr int WARPS = B_::WARPS, THREADS = B_::THREADS;
    static constexpr int CTAS_PER_SM = B_::CTAS_PER_SM;
    static constexpr int Q = B_::Q;
    static constexpr int STAGES = 8;                   // ring depth per warp (positions): a stage is 5 n floats
    static constexpr int STAGE_FLOATS = 5 * N;         // coefficient rows [N][4], then the vector [N]
    // weights in shared memory, laid out so that what a lane (g,t) needs from one row is contiguous:
    //   forward: row i holds, for t = 0..3, {W[i][8kk+2t], W[i][8kk+2t+1]} for kk = 0..NT-1
    //   reverse: row i holds, for g = 0..7, W[i][8nn+g] for nn = 0..NT-1
    // (128-bit reads at n = 32); the row stride makes the reads of a quarter- or half-warp fall in distinct banks
    static constexpr int WS = N + (N == 32 ? 4 : (REV ? 4 : 0));
    static constexpr int RES_WARPS = B_::RES_WARPS;
    static constexpr int PEND = B_::PEND;
    static constexpr int SM_WORK = Q * PEND + WARPS * N + N + 16 + 3 * N * WS + WARPS * STAGES * STAGE_FLOATS;
    static constexpr int SM_RES = B_::SM_RES;
    static constexpr int SM_FLOATS = SM_WORK > SM_RES ? SM_WORK : SM_RES;
    static constexpr size_t SMEM = SM_FLOATS * sizeof(float) + 128;
    static constexpr int MAX_SEQ_PER_WARP = B_::MAX_SEQ_PER_WARP;
    static_assert(STAGES * STAGE_FLOATS >= AGG, "the last warp's aggregate is parked in its ring");
};

// The lane's pieces of J_t, jp[nn][kk] = {J[8nn+g][8kk+2t], J[8nn+g][8kk+2t+1]}, from the staged
// coefficient rows cf[i] = {k_r, a_z, k_n, z}_i and the weights in shared memory.
// reverse form: jp[nn][kk] = {J[8kk+2t][8nn+g], J[8kk+2t+1][8nn+g]} (the operand is J, not its transpose)
template <int N>
__device__ __forceinline__ void gen_pieces_rev(float (&jp)[N / 8][N / 8][2], const float *stage, const float *sW,
                                               int g, int t, bool d0, bool d1)
{
    constexpr int NT = N / 8, WS = WarpNF<N, true>::WS;
#pragma unroll
    for (int kk = 0; kk < NT; ++kk) {
#pragma unroll
        for (int e = 0; e < 2; ++e) {
            const int row = 8 * kk + 2 * t + e;
            const float4 cf = *reinterpret_cast<const float4 *>(stage + 4 * row);
            const float *wrow = sW + row * WS + g * NT;
            float wr[NT], wz[NT], wn[NT];
            if constexpr (NT == 4) {
                const float4 r4 = *reinterpret_cast<const float4 *>(wrow);
                const float4 z4 = *reinterpret_cast<const float4 *>(wrow + N * WS);
                const float4 n4 = *reinterpret_cast<const float4 *>(wrow + 2 * N * WS);
                wr[0] = r4.x; wr[1] = r4.y; wr[2] = r4.z; wr[3] = r4.w;
                wz[0] = z4.x; wz[1] = z4.y; wz[2] = z4.z; wz[3] = z4.w;
                wn[0] = n4.x; wn[1] = n4.y; wn[2] = n4.z; wn[3] = n4.w;
            } else {
                const float2 r2 = *reinterpret_cast<const float2 *>(wrow);
                const float2 z2 = *reinterpret_cast<const float2 *>(wrow + N * WS);
                const float2 n2 = *reinterpret_cast<const float2 *>(wrow + 2 * N * WS);
                wr[0] = r2.x; wr[1] = r2.y; wz[0] = z2.x; wz[1] = z2.y; wn[0] = n2.x; wn[1] = n2.y;
            }
#pragma unroll
            for (int nn = 0; nn < NT; ++nn) {
                float v = fmaf(cf.x, wr[nn], fmaf(cf.y, wz[nn], cf.z * wn[nn]));
                if (nn == kk) v += (e == 0 ? d0 : d1) ? cf.w : 0.0f;
                jp[nn][kk][e] = v;
            }
        }
    }
}

template <int N>
__device__ __forceinline__ void gen_pieces(float (&jp)[N / 8][N / 8][2], const float *stage, const float *sW,
                                           int g, int t, bool d0, bool d1)
{
    constexpr int NT = N / 8, WS = WarpNF<N>::WS;
#pragma unroll
    for (int nn = 0; nn < NT; ++nn) {
        const float4 cf = *reinterpret_cast<const float4 *>(stage + 4 * (8 * nn + g));
        const float *wrow = sW + (8 * nn + g) * WS + t * 2 * NT;
        float wr[2 * NT], wz[2 * NT], wn[2 * NT];
#pragma unroll
        for (int v = 0; v < 2 * NT / 4; ++v) {
            const float4 r4 = reinterpret_cast<const float4 *>(wrow)[v];
            const float4 z4 = reinterpret_cast<const float4 *>(wrow + N * WS)[v];
            const float4 n4 = reinterpret_cast<const float4 *>(wrow + 2 * N * WS)[v];
            wr[4 * v] = r4.x; wr[4 * v + 1] = r4.y; wr[4 * v + 2] = r4.z; wr[4 * v + 3] = r4.w;
            wz[4 * v] = z4.x; wz[4 * v + 1] = z4.y; wz[4 * v + 2] = z4.z; wz[4 * v + 3] = z4.w;
            wn[4 * v] = n4.x; wn[4 * v + 1] = n4.y; wn[4 * v + 2] = n4.z; wn[4 * v + 3] = n4.w;
        }
        const float2 cx = make_float2(cf.x, cf.x), cy = make_float2(cf.y, cf.y), cz = make_float2(cf.z, cf.z);
#pragma unroll
        for (int kk = 0; kk < NT; ++kk) {
            float2 v = ffma2(cx, make_float2(wr[2 * kk], wr[2 * kk + 1]),
                             ffma2(cy, make_float2(wz[2 * kk], wz[2 * kk + 1]), fmul2(cz, make_float2(wn[2 * kk], wn[2 * kk + 1]))));
            if (nn == kk) { v.x += d0 ? cf.w : 0.0f; v.y += d1 ? cf.w : 0.0f; }
            jp[nn][kk][0] = v.x; jp[nn][kk][1] = v.y;
        }
    }
}

template <int N, bool REV>
__global__ void __launch_bounds__(WarpNF<N, REV>::THREADS, WarpNF<N, REV>::CTAS_PER_SM) scan_warpnf_kernel(ScanArgs a, OnePassWs w)
{
    using C = WarpNF<N, REV>;
    constexpr int NN = C::NN, AGG = C::AGG, NT = C::NT, MT = C::MT, WARPS = C::WARPS, Q = C::Q;
    pdl_prologue();
    if (loop_ended(a.st)) return;

    extern __shared__ __align__(16) float smem_raw[];
    float *sm = (float *)(((uintptr_t)smem_raw + 127) & ~(uintptr_t)127);
    float *pend = sm;                          // Q x warp aggregates (A row-major, then beta)
    float *wstart = pend + Q * C::PEND;        // WARPS x N states entering each warp chain
    float *ystart = wstart + WARPS * N;
    float *sW = ystart + N + 16;               // W_hr, W_hz, W_hn with rows padded to WS floats
    float *ring_all = sW + 3 * N * C::WS;      // WARPS x STAGES x (coefficients [N][4], vector [N])
    __shared__ int s_kind, s_seq, s_c, s_slot, s_abort, s_role;

    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const int g = lane >> 2, t = lane & 3;
    const int T = a.T;
    constexpr int S = C::STAGES;
    float *ring = ring_all + warp * S * C::STAGE_FLOATS;
    const int SW = w.sw, L = WARPS * SW;
    for (int i = tid; i < 3 * NN; i += C::THREADS) {
        const int col = i % N, kk = col >> 3, tt = (col & 7) >> 1, e = col & 1;
        if (!REV) sW[(i / N) * C::WS + tt * 2 * NT + 2 * kk + e] = a.Wh[i];
        else sW[(i / N) * C::WS + (col & 7) * NT + kk] = a.Wh[i];
    }
    const bool d0 = g == 2 * t, d1 = g == 2 * t + 1;      // this lane's pieces touch the diagonal where nn == kk

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
        const float *Cseq = a.J + (size_t)seq * T * 4 * N;      // coefficient rows {k_r, a_z, k_n, z}[N] per position
        const float *bseq = a.b + (size_t)seq * T * N;
        // scan position s: forward matrix J[s], vector at s; reverse matrix J[T-s] (identity at s = 0:
        // coefficient rows {0,0,0,1}), vector at T-1-s
        auto pos_t = [&](int s) -> size_t { return REV ? (size_t)(T - 1 - s) : (size_t)s; };
        // chain position q -> ring stage q % S (one commit group per call, also past the end)
        auto issue = [&](int q) {
            const int s = sbase + q;
            if (q < cnt) {
                float *dst = ring + (q % S) * C::STAGE_FLOATS;
                const float *cs = Cseq + (REV ? (size_t)(T - s) : (size_t)s) * 4 * N, *bs = bseq + pos_t(s) * N;
                const bool ident = REV && s == 0;
#pragma unroll
                for (int u = 0; u < (5 * N / 4 + 31) / 32; ++u) {
                    const int j = lane + 32 * u;
                    if (j < N) {
                        if (ident) *reinterpret_cast<float4 *>(dst + 4 * j) = make_float4(0.0f, 0.0f, 0.0f, 1.0f);
                        else cp_async16(dst + 4 * j, cs + 4 * j);
                    } else if (j < N + N / 4) cp_async16(dst + 4 * j, bs + 4 * (j - N));
                }
            }
            cp_async_commit();
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
                if constexpr (REV) gen_pieces_rev<N>(jp, Ms, sW, g, t, d0, d1); else gen_pieces<N>(jp, Ms, sW, g, t, d0, d1);
#pragma unroll
                for (int nn = 0; nn < NT; ++nn) bg[nn] = Ms[4 * N + 8 * nn + g];
                if constexpr (REV) chain_step_n<N>(acc, jp); else chain_step_n1<N>(acc, jp);
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
                    if constexpr (REV) chain_step_n<N>(acc, jp); else chain_step_n1<N>(acc, jp);
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
                if constexpr (REV) gen_pieces_rev<N>(jp, Ms, sW, g, t, d0, d1); else gen_pieces<N>(jp, Ms, sW, g, t, d0, d1);
                const size_t vb = ((size_t)seq * T + pos_t(s)) * N;
#pragma unroll
                for (int nn = 0; nn < NT; ++nn) bg[nn] = Ms[4 * N + 8 * nn + g];
                matvec_step<N>(yv, jp, bg, ynew, t);
                if (t == 0) {
#pragma unroll
                    for (int nn = 0; nn < NT; ++nn) {
                        if constexpr (!REV) {
                            // Newton-update form: the scanned quantity is the update; y = y_old + update
                            // (err is taken from the two stored iterates, as the diagnostics kernel does)
                            const float yo = __ldg(a.yold + vb + 8 * nn + g), yn = yo + ynew[nn];
                            mb = max(mb, absdiff_bits(yn, yo));
                            a.y[vb + 8 * nn + g] = yn;
                        } else {
                            if (a.yold) mb = max(mb, absdiff_bits(ynew[nn], __ldg(a.yold + vb + 8 * nn + g)));
                            a.y[vb + 8 * nn + g] = ynew[nn];
                        }
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
