// The scan inside deer_gru_eval for n = 64 (J generated from coefficient rows), Newton-update form, two launches
// as for n = 16, 32 (scan_fused_fwd.cuh): chunk reduce + carries, then the lockstep replay of all chains.
//
// A 64 x 64 running product with its 12,288 weights does not fit one warp, so a chain is advanced by a CTA of
// four warps, and a tile is a single chain (the resolver CTAs, those of scan_cta64.cuh, walk the chain
// aggregates directly: no prefix aggregates).  Per position:
//   * warp w builds rows 16w .. 16w+15 of J_t from the staged coefficient rows and ITS share of W_h, which it
//     keeps in registers for the whole launch as bf16 pairs (48 per lane), in packed bf16 arithmetic (the result
//     is the m16n8k16 B operand as it stands), and writes them to shared memory (8 KB per position,
//     double-buffered); it also advances its 16 components of beta: beta^T J_t^T for its columns is eight more
//     MMAs on the fragments it has just built (beta exchanged through shared memory);
//   * every warp multiplies ITS 16 rows of X = P^T by J_t^T: 32 bf16 MMAs with the accumulator tiles of X as the
//     A operand as they stand (fp32 accumulate, 8 independent accumulators).
// The rows of position q + 1 do not depend on X: they are built in the same loop body as the products of position q,
// so a position costs ONE CTA barrier and the two kinds of work fill each other's gaps.
// The replay kernel is scan_fused_apply_kernel<64>: W_h^T as the B operand from shared memory (48 KB: it does
// not fit the registers of one warp), TF32.
#pragma once
#include "scan_cta64.cuh"
#include "scan_fused_fwd.cuh"

namespace deer {

template <> struct FusedFwd<64> {
    static constexpr int N = 64, NN = N * N, AGG = NN + N, NT = 8;
    static constexpr int WARPS = 1;                    // chains per tile: the apply kernel needs no prefix aggregates
    static constexpr int R_WARPS = 4, THREADS = 128;   // reduce kernel: four warps advance one chain
    static constexpr int L = Cta64::L;                 // positions per chain / tile
    static constexpr int STAGES = 6;                   // CTA-wide ring depth (positions)
    static constexpr int STAGE_FLOATS = 5 * N;         // coefficient rows [N][4], then the residual [N]
    static constexpr int JB_WORDS = NT * 2 * 32 * 4;   // bf16 B fragments of one position: [nn][half][lane][4 words]
    static constexpr int RES_WARPS = Cta64::RES_WARPS, MAX_SEQ_PER_WARP = Cta64::MAX_SEQ_PER_WARP;
    static constexpr int SM_WORK = STAGES * STAGE_FLOATS + 2 * JB_WORDS + 2 * N + 16;
    static constexpr int RES_SLOTS = 4;                // tile aggregates a resolver CTA stages, shared by its resolving warps
    static constexpr int SM_RES = RES_SLOTS * AGG + RES_WARPS * N;
    static constexpr int SM_FLOATS = SM_WORK > SM_RES ? SM_WORK : SM_RES;
    static constexpr size_t SMEM = SM_FLOATS * sizeof(float) + 128;
    // apply kernel
    static constexpr int ROWS = 16;
    static constexpr int A_WARPS = 2, A_THREADS = 64, A_STAGES = 3;
    static constexpr int ROW_FLOATS = 6 * N + 4;
    static constexpr int STAGE_A = ROWS * ROW_FLOATS;
    static constexpr bool W_SMEM = true;
    static constexpr size_t A_SMEM = sizeof(float) * (A_WARPS * A_STAGES * STAGE_A + A_WARPS * ROWS * N + 2 * NT * 3 * NT * 32) + 128;
};

__global__ void __launch_bounds__(FusedFwd<64>::THREADS, 3) scan_fused_reduce64_kernel(ScanArgs a, OnePassWs w)
{
    using C = FusedFwd<64>;
    constexpr int N = C::N, NN = C::NN, AGG = C::AGG, NT = C::NT, S = C::STAGES, L = C::L;
    pdl_prologue();
    if (loop_ended(a.st)) return;

    extern __shared__ __align__(16) float smem_raw[];
    float *sm = (float *)(((uintptr_t)smem_raw + 127) & ~(uintptr_t)127);
    float *ring = sm;                                              // S x (coefficients [N][4], residual [N])
    uint4 *Jb = reinterpret_cast<uint4 *>(ring + S * C::STAGE_FLOATS);   // 2 x [nn][half][lane] (4 words each)
    float *beta = reinterpret_cast<float *>(Jb) + 2 * C::JB_WORDS;  // 2 x [N]
    __shared__ int s_seq, s_c, s_role;

    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const int g = lane >> 2, t = lane & 3;
    const int T = a.T;

    // this warp's rows of J: i = 8 (2 warp + h) + g, h = 0, 1; its weights for them, by B-operand piece (j, e):
    // columns 16 j + 8 e + 2t, + 1
    unsigned wR[2][4][2], wZ[2][4][2], wN[2][4][2];
#pragma unroll
    for (int h = 0; h < 2; ++h)
#pragma unroll
        for (int j = 0; j < 4; ++j)
#pragma unroll
            for (int e = 0; e < 2; ++e) {
                const float *wp = a.Wh + (size_t)(8 * (2 * warp + h) + g) * N + 16 * j + 8 * e + 2 * t;
                const float2 r2 = __ldg(reinterpret_cast<const float2 *>(wp));
                const float2 z2 = __ldg(reinterpret_cast<const float2 *>(wp + NN));
                const float2 n2 = __ldg(reinterpret_cast<const float2 *>(wp + 2 * NN));
                wR[h][j][e] = pack_bf16(r2.x, r2.y); wZ[h][j][e] = pack_bf16(z2.x, z2.y); wN[h][j][e] = pack_bf16(n2.x, n2.y);
            }
    const bool d0 = g == 2 * t, d1 = g == 2 * t + 1;      // the piece (j, e) = ((2 warp + h) / 2, (2 warp + h) % 2) holds the diagonal

    if (tid == 0) s_role = (int)atomicAdd(&a.st->role_counter, 1u);
    __syncthreads();
    if (s_role < w.resolvers) {
        if (warp < w.res_warps)
            resolver64(a, w, sm, C::RES_SLOTS, s_role * w.res_warps + warp, w.resolvers * w.res_warps, lane);
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
    unsigned next_id = 0;
    if (tid == 0) next_id = atomicAdd(&a.st->tile_counter, 1u);

    for (;;) {
        __syncthreads();
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
        const int sbase = c * L;
        const int cnt = min(L, T - sbase);
        const size_t tile_index = (size_t)seq * w.nch + c;
        const float *Cseq = a.J + ((size_t)seq * T + sbase) * 4 * N;
        const float *bseq = a.b + ((size_t)seq * T + sbase) * N;
        // CTA-wide ring: 80 pieces of 16 bytes per position (always one commit group per thread and call)
        auto issue = [&](int q) {
            if (q < cnt && tid < 5 * N / 4) {
                float *dst = ring + (q % S) * C::STAGE_FLOATS;
                if (tid < N) cp_async16(dst + 4 * tid, Cseq + (size_t)q * 4 * N + 4 * tid);
                else cp_async16(dst + 4 * tid, bseq + (size_t)q * N + 4 * (tid - N));
            }
            cp_async_commit();
        };

        // X = identity: this warp's rows 16 warp + g (+8), column tiles nn
        float acc[NT][4];
#pragma unroll
        for (int nn = 0; nn < NT; ++nn) {
            const int r = 16 * warp + g, cc = 8 * nn + 2 * t;
            acc[nn][0] = (r == cc) ? 1.0f : 0.0f;     acc[nn][1] = (r == cc + 1) ? 1.0f : 0.0f;
            acc[nn][2] = (r + 8 == cc) ? 1.0f : 0.0f; acc[nn][3] = (r + 8 == cc + 1) ? 1.0f : 0.0f;
        }
        if (tid < N) beta[tid] = 0.0f;
#pragma unroll
        for (int q = 0; q < S - 1; ++q) issue(q);

        // this warp's 16 rows of J_p (bf16 B fragments to shared memory) and its 16 components of beta_{p+1} = J_p beta_p + r_p
        auto build = [&](int p) {
            const float *Ms = ring + (p % S) * C::STAGE_FLOATS;
            const float *bin = beta + (p & 1) * N;
            float *bout = beta + ((p + 1) & 1) * N;
            uint4 *Jp = Jb + (p & 1) * (C::JB_WORDS / 4);
            // beta^T as the live row of an A operand (lanes g == 0), one k block of 16 per j
            unsigned ab[4][2];
#pragma unroll
            for (int j = 0; j < 4; ++j) {
                const float2 lo = *reinterpret_cast<const float2 *>(bin + 16 * j + 2 * t);
                const float2 hi = *reinterpret_cast<const float2 *>(bin + 16 * j + 8 + 2 * t);
                ab[j][0] = g == 0 ? pack_bf16(lo.x, lo.y) : 0u;
                ab[j][1] = g == 0 ? pack_bf16(hi.x, hi.y) : 0u;
            }
#pragma unroll
            for (int h = 0; h < 2; ++h) {
                const int nn = 2 * warp + h, i = 8 * nn + g;
                const float4 cf = *reinterpret_cast<const float4 *>(Ms + 4 * i);
                const unsigned cr = pack_bf16(cf.x, cf.x), cz = pack_bf16(cf.y, cf.y), cn = pack_bf16(cf.z, cf.z);
                const unsigned zd = pack_bf16(d0 ? cf.w : 0.0f, d1 ? cf.w : 0.0f);
                unsigned words[4][2];
#pragma unroll
                for (int j = 0; j < 4; ++j)
#pragma unroll
                    for (int e = 0; e < 2; ++e) words[j][e] = hmul2_bf16(cn, wN[h][j][e]);
#pragma unroll
                for (int j = 0; j < 4; ++j)
#pragma unroll
                    for (int e = 0; e < 2; ++e) words[j][e] = hfma2_bf16(cz, wZ[h][j][e], words[j][e]);
#pragma unroll
                for (int j = 0; j < 4; ++j)
#pragma unroll
                    for (int e = 0; e < 2; ++e) {
                        words[j][e] = hfma2_bf16(cr, wR[h][j][e], words[j][e]);
                        if (2 * j + e == nn) words[j][e] = hadd2_bf16(words[j][e], zd);
                    }
                Jp[(nn * 2 + 0) * 32 + lane] = make_uint4(words[0][0], words[0][1], words[1][0], words[1][1]);
                Jp[(nn * 2 + 1) * 32 + lane] = make_uint4(words[2][0], words[2][1], words[3][0], words[3][1]);
                float cb[4] = {0.0f, 0.0f, 0.0f, 0.0f};
#pragma unroll
                for (int j = 0; j < 4; ++j) {
                    const unsigned af[4] = {ab[j][0], 0u, ab[j][1], 0u};
                    mma_bf16(cb, af, words[j], cb);
                }
                if (g == 0) {
                    const float2 r2 = *reinterpret_cast<const float2 *>(Ms + 4 * N + 8 * nn + 2 * t);
                    *reinterpret_cast<float2 *>(bout + 8 * nn + 2 * t) = make_float2(cb[0] + r2.x, cb[1] + r2.y);
                }
            }
        };
        cp_async_wait_n<S - 2>();
        __syncthreads();                       // stage 0 and beta_0 visible
        if (cnt > 0) build(0);

#pragma unroll 1
        for (int q = 0; q < cnt; ++q) {
            cp_async_wait_n<S - 3>();
            __syncthreads();                   // J_q, beta_{q+1} and stage q + 1 visible to all; the buffers of position q - 1 are free
            issue(q + S - 1);
            const uint4 *Jq = Jb + (q & 1) * (C::JB_WORDS / 4);
            // ---- X <- X J_q^T for this warp's 16 rows: accumulator tiles 2j, 2j+1 are the A operand of block j
            unsigned af[4][4];
#pragma unroll
            for (int j = 0; j < 4; ++j) {
                af[j][0] = pack_bf16(acc[2 * j][0], acc[2 * j][1]);
                af[j][1] = pack_bf16(acc[2 * j][2], acc[2 * j][3]);
                af[j][2] = pack_bf16(acc[2 * j + 1][0], acc[2 * j + 1][1]);
                af[j][3] = pack_bf16(acc[2 * j + 1][2], acc[2 * j + 1][3]);
            }
#pragma unroll
            for (int nn = 0; nn < NT; ++nn) { acc[nn][0] = 0.0f; acc[nn][1] = 0.0f; acc[nn][2] = 0.0f; acc[nn][3] = 0.0f; }
#pragma unroll
            for (int half = 0; half < 2; ++half) {
                uint4 bw[NT];
#pragma unroll
                for (int nn = 0; nn < NT; ++nn) bw[nn] = Jq[(nn * 2 + half) * 32 + lane];
#pragma unroll
                for (int nn = 0; nn < NT; ++nn) {
                    const unsigned bf[2] = {bw[nn].x, bw[nn].y};
                    mma_bf16(acc[nn], af[2 * half], bf, acc[nn]);
                }
#pragma unroll
                for (int nn = 0; nn < NT; ++nn) {
                    const unsigned bf[2] = {bw[nn].z, bw[nn].w};
                    mma_bf16(acc[nn], af[2 * half + 1], bf, acc[nn]);
                }
            }
            // ---- the rows of the next position and beta_{q+2}, while those MMAs are in flight
            if (q + 1 < cnt) build(q + 1);
        }
        cp_async_wait_n<0>();
        __syncthreads();
        // ---- the chain's aggregate: P[c][r] = X[r][c] (row-major), then beta; publish
        {
            float *dst = w.aggs + tile_index * AGG;
            const int r = 16 * warp + g;
#pragma unroll
            for (int nn = 0; nn < NT; ++nn) {
                const int cc = 8 * nn + 2 * t;
                dst[cc * N + r] = acc[nn][0];
                dst[(cc + 1) * N + r] = acc[nn][1];
                dst[cc * N + r + 8] = acc[nn][2];
                dst[(cc + 1) * N + r + 8] = acc[nn][3];
            }
            if (tid < N) dst[NN + tid] = beta[(cnt & 1) * N + tid];
        }
        __threadfence();
        __syncthreads();
        if (tid == 0) st_release_u32(w.flags + tile_index, 1u);
    }
    __syncthreads();
    if (tid == 0) scan_epilogue(a.st, false);
}

}  // namespace deer
