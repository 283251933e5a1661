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
// The replay kernel is scan_fused_apply64_kernel below: W_h^T as the B operand from shared memory (48 KB: it does
// not fit the registers of one warp), TF32, two warps per group of 16 chains.
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
    static constexpr int ROW_FLOATS = 6 * N + 4;
    static constexpr int STAGE_A = ROWS * ROW_FLOATS;
    // pair-split replay (scan_fused_apply64_kernel): two warps share a group of 16 chains, each with half of the state
    // columns; a CTA holds P_PAIRS pairs
    static constexpr int P_PAIRS = 2, P_THREADS = 64 * P_PAIRS, P_STAGES = 3;
    static constexpr int P_XCH = 2 * NT * 32 * 4;      // floats of a pair's state exchange (two buffers of [NT][32] float4)
    static constexpr int P_PAIR_FLOATS = P_STAGES * STAGE_A + P_XCH;
    static constexpr size_t P_SMEM = sizeof(float) * (P_PAIRS * P_PAIR_FLOATS + 2 * NT * 3 * NT * 32) + 128;
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


// The replay for n = 64 with TWO warps per group of 16 chains.  A step of the 16-chain replay is 192 MMAs: issued by one
// warp they keep one sub-partition busy and shared memory has room for two such warps per SM only.  Here warp h of a
// pair multiplies the full state D [16, 64] into ITS 96 of the 192 output columns (the r, z and candidate columns of the
// state columns 32h .. 32h+31), runs the elementwise epilogue for those state columns, and the two halves of the new D
// are exchanged through shared memory (one 64-thread barrier per step, double-buffered): the same ring serves the pair,
// so four warps per SM share the memory two needed.  Staging, epilogue arithmetic and the error word are those of
// scan_fused_apply_kernel; a tile is one chain (entering states straight from the resolvers' words).
__global__ void __launch_bounds__(FusedFwd<64>::P_THREADS) scan_fused_apply64_kernel(ScanArgs a, OnePassWs w)
{
    using C = FusedFwd<64>;
    constexpr int N = 64, NT = C::NT, HT = NT / 2, ROWS = C::ROWS, RF = C::ROW_FLOATS, S = C::P_STAGES;
    pdl_prologue();
    if (loop_ended(a.st)) return;

    extern __shared__ __align__(16) float smem_raw[];
    float *sm = (float *)(((uintptr_t)smem_raw + 127) & ~(uintptr_t)127);
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const int pair = warp >> 1, hw = warp & 1;
    const int g = lane >> 2, t = lane & 3;
    float *ring = sm + pair * C::P_PAIR_FLOATS;
    float4 *xch = reinterpret_cast<float4 *>(ring + S * C::STAGE_A);        // [2][NT][32]
    float *yin = ring;                                                       // entering states: stage 0, before the ring is in use
    float2 *sWf = reinterpret_cast<float2 *>(sm + C::P_PAIRS * C::P_PAIR_FLOATS);   // [kk][nn][lane]
    for (int idx = tid; idx < NT * 3 * NT * 32; idx += C::P_THREADS) {
        const int l = idx & 31, nn = (idx >> 5) % (3 * NT), kk = (idx >> 5) / (3 * NT);
        sWf[idx] = __ldg(reinterpret_cast<const float2 *>(a.Wh + (size_t)(8 * nn + (l >> 2)) * N + 8 * kk + 2 * (l & 3)));
    }
    __syncthreads();
    auto pair_sync = [&]() { asm volatile("bar.sync %0, 64;" ::"r"(1 + pair) : "memory"); };
    const float2 *sWh = sWf + HT * hw * 32 + lane;     // this warp's column blocks of every gate

    const int T = a.T, SW = w.sw;
    const long long nchain = (T + SW - 1) / SW;
    const long long total = (long long)a.B * nchain;
    const long long groups = (total + ROWS - 1) / ROWS;
    unsigned mb = 0;
    unsigned it0 = 0;

    for (long long grp = (long long)blockIdx.x * C::P_PAIRS + pair; grp < groups; grp += (long long)gridDim.x * C::P_PAIRS) {
        const int row = lane & 15;
        const long long gid = grp * ROWS + row;
        const bool rv = gid < total;
        const long long seq = rv ? gid / nchain : 0;
        const int q = rv ? (int)(gid - seq * nchain) : 0;
        const int len = rv ? min(SW, T - q * SW) : 0;
        const size_t e0 = (size_t)seq * T + (size_t)q * SW;
        const size_t tile_index = (size_t)seq * w.nch + q;
        int maxlen = len;
#pragma unroll
        for (int o = 8; o > 0; o >>= 1) maxlen = max(maxlen, __shfl_xor_sync(0xffffffffu, maxlen, o));

        pair_sync();                           // the previous group's last stage and exchange buffers are no longer read
        // entering states of the 16 chains (warp h fetches rows 8h .. 8h+7)
        for (int r = 8 * hw; r < 8 * hw + 8; ++r) {
            const int vr = __shfl_sync(0xffffffffu, (int)rv, r);
            const unsigned long long tix = __shfl_sync(0xffffffffu, (unsigned long long)tile_index, r);
            for (int c = lane; c < N; c += 32)
                yin[r * N + c] = vr ? __uint_as_float((unsigned)(ld_relaxed_u64(w.starts + tix * N + c) & 0xffffffffull)) : 0.0f;
        }
        pair_sync();
        float d[NT][4];
#pragma unroll
        for (int nn = 0; nn < NT; ++nn) {
            const float2 lo = *reinterpret_cast<const float2 *>(yin + g * N + 8 * nn + 2 * t);
            const float2 hi = *reinterpret_cast<const float2 *>(yin + (g + 8) * N + 8 * nn + 2 * t);
            d[nn][0] = lo.x; d[nn][1] = lo.y; d[nn][2] = hi.x; d[nn][3] = hi.y;
        }
        pair_sync();                           // yin (stage 0) may be overwritten by the ring from here on
        const int len_lo = __shfl_sync(0xffffffffu, len, g), len_hi = __shfl_sync(0xffffffffu, len, g + 8);
        const unsigned long long e_lo = __shfl_sync(0xffffffffu, (unsigned long long)e0, g);
        const unsigned long long e_hi = __shfl_sync(0xffffffffu, (unsigned long long)e0, g + 8);
        float *yp[2] = {a.y + e_lo * N + 2 * t, a.y + e_hi * N + 2 * t};
        const int lens[2] = {len_lo, len_hi};

        // staging: eight lanes copy 128 contiguous bytes of a row; warp h serves the rows 8h + 4k + (lane >> 3), k = 0, 1
        const int rsub = lane >> 3, cpos = 4 * (lane & 7);
        unsigned long long e0q[2];
        int lenq[2];
#pragma unroll
        for (int k = 0; k < 2; ++k) {
            e0q[k] = __shfl_sync(0xffffffffu, (unsigned long long)e0, 8 * hw + 4 * k + rsub);
            lenq[k] = __shfl_sync(0xffffffffu, len, 8 * hw + 4 * k + rsub);
        }
        auto issue = [&](int s) {
            float *stg_dst = ring + ((it0 + (unsigned)s) % S) * C::STAGE_A + (8 * hw + rsub) * RF + cpos;
#pragma unroll
            for (int k = 0; k < 2; ++k) {
                if (s < lenq[k]) {
                    float *dst = stg_dst + 4 * k * RF;
                    const size_t e = (size_t)e0q[k] + (size_t)s;
                    const float *sc = a.J + e * 4 * N + cpos, *sr = a.b + e * N + cpos, *so = a.yold + e * N + cpos;
#pragma unroll
                    for (int j = 0; j < N / 8; ++j) cp_async16(dst + 32 * j, sc + 32 * j);
#pragma unroll
                    for (int j = 0; j < N / 32; ++j) {
                        cp_async16(dst + 4 * N + 32 * j, sr + 32 * j);
                        cp_async16(dst + 5 * N + 32 * j, so + 32 * j);
                    }
                }
            }
            cp_async_commit();
        };
#pragma unroll
        for (int s = 0; s < S - 1; ++s) issue(s);
        cp_async_wait_n<S - 2>();
        pair_sync();                           // step 0 landed for both warps

#pragma unroll 1
        for (int s = 0; s < maxlen; ++s) {
            issue(s + S - 1);                  // into the stage of step s - 1, which both warps left before the last barrier
            const unsigned stg = (it0 + (unsigned)s) % S;
            // U = D W_h^T for this warp's 96 columns: blocks 4h .. 4h+3 of each gate
            float U[3 * HT][4];
#pragma unroll
            for (int j = 0; j < 3 * HT; ++j) { U[j][0] = 0.0f; U[j][1] = 0.0f; U[j][2] = 0.0f; U[j][3] = 0.0f; }
#pragma unroll
            for (int kk = 0; kk < NT; ++kk) {
                const unsigned af[4] = {__float_as_uint(d[kk][0]), __float_as_uint(d[kk][2]), __float_as_uint(d[kk][1]),
                                        __float_as_uint(d[kk][3])};
#pragma unroll
                for (int j = 0; j < 3 * HT; ++j) {
                    const float2 b2 = sWh[(kk * 3 * NT + (j / HT) * NT + (j % HT)) * 32];
                    const unsigned bf[2] = {__float_as_uint(b2.x), __float_as_uint(b2.y)};
                    mma_tf32(U[j], af, bf, U[j]);
                }
            }
            const float *st = ring + stg * C::STAGE_A;
            float dn[HT][4];                   // this warp's state columns (rows past their chain's end keep their value)
#pragma unroll
            for (int jj = 0; jj < HT; ++jj)
#pragma unroll
                for (int i = 0; i < 4; ++i) dn[jj][i] = hw ? d[HT + jj][i] : d[jj][i];
#pragma unroll
            for (int h = 0; h < 2; ++h) {
                if (s < lens[h]) {
                    const float *rs = st + (g + 8 * h) * RF;
#pragma unroll
                    for (int jj = 0; jj < HT; ++jj) {
                        const int nn = HT * hw + jj;
                        const int col = 8 * nn + 2 * t;
                        const float4 c0 = *reinterpret_cast<const float4 *>(rs + 4 * col);
                        const float4 c1 = *reinterpret_cast<const float4 *>(rs + 4 * col + 4);
                        const float2 r2 = *reinterpret_cast<const float2 *>(rs + 4 * N + col);
                        const float2 yo = *reinterpret_cast<const float2 *>(rs + 5 * N + col);
                        float dx = fmaf(c0.w, dn[jj][2 * h], r2.x), dy = fmaf(c1.w, dn[jj][2 * h + 1], r2.y);
                        dx = fmaf(c0.x, U[jj][2 * h], dx);              dy = fmaf(c1.x, U[jj][2 * h + 1], dy);
                        dx = fmaf(c0.y, U[HT + jj][2 * h], dx);         dy = fmaf(c1.y, U[HT + jj][2 * h + 1], dy);
                        dx = fmaf(c0.z, U[2 * HT + jj][2 * h], dx);     dy = fmaf(c1.z, U[2 * HT + jj][2 * h + 1], dy);
                        dn[jj][2 * h] = dx; dn[jj][2 * h + 1] = dy;
                        const float2 yn = make_float2(yo.x + dx, yo.y + dy);
                        mb = max(mb, absdiff_bits(yn.x, yo.x));
                        mb = max(mb, absdiff_bits(yn.y, yo.y));
                        *reinterpret_cast<float2 *>(yp[h] + (size_t)s * N + 8 * nn) = yn;
                    }
                }
            }
            // the new state: this warp's column blocks out, the partner's in
            float4 *xb = xch + (s & 1) * NT * 32;
#pragma unroll
            for (int jj = 0; jj < HT; ++jj) xb[(HT * hw + jj) * 32 + lane] = make_float4(dn[jj][0], dn[jj][1], dn[jj][2], dn[jj][3]);
            cp_async_wait_n<S - 2>();          // this warp's copies of step s + 1
            pair_sync();
#pragma unroll
            for (int kk = 0; kk < NT; ++kk) {
                const float4 v = xb[kk * 32 + lane];
                d[kk][0] = v.x; d[kk][1] = v.y; d[kk][2] = v.z; d[kk][3] = v.w;
            }
        }
        cp_async_wait_n<0>();
        it0 += (unsigned)maxlen;
    }
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) mb = max(mb, __shfl_xor_sync(0xffffffffu, mb, o));
    if (lane == 0 && mb) { atomicMax(&a.st->err_bits, mb); __threadfence(); }
    __syncthreads();
    if (tid == 0) scan_epilogue(a.st, true);
}

}  // namespace deer
