// Single-pass scan for n = 64: one CTA (two warps) per chain, chain product on tensor cores.
//
// A 64 x 64 running product does not fit one warp's registers, so a tile is a single chain that
// the CTA's two warps advance together: warp w keeps rows 32w .. 32w+31 of X = P^T in 2 x 8
// accumulator fragments and both multiply by the same matrix,
//       X <- X * M,   M = J_t^T (forward)  or  J_{t+1} (reverse),
// 2 x 8 x 8 MMAs (m16n8k8) per warp and position, each issued three times on hi/lo TF32 splits.
// The matrices of the tile stream through a shared-memory ring filled with 16-byte cp.async
// copies; rows are padded (by 8 floats forward, 4 in reverse) so that the B-operand reads (8-byte
// pieces of a row forward, scalars of a column in reverse) and the row / column reads of the
// mat-vec are all free of bank conflicts.  beta (the state reached from
// zero) is carried by an fp32 mat-vec chain, thread r owning component r; the same routine
// replays the tile from its true entering state in the B item.
// Tiles, items, resolvers, flags and bounded waits are those of scan_onepass.cuh.
#pragma once
#include "scan_warpn.cuh"

namespace deer {

struct Cta64 {
    static constexpr int N = 64, NN = N * N, AGG = NN + N;
    static constexpr int NT = 8;                       // 8-wide column / contraction blocks
    static constexpr int MT = 2;                       // 16-high row blocks of X per warp
    static constexpr int WARPS = 2, THREADS = 64;
    static constexpr int L = 64;                       // positions per tile
    static constexpr int Q = 2;                        // pending tiles per CTA
    static constexpr int STAGES = 3;                   // ring depth (positions)
    static constexpr int STAGE_FLOATS = N * (N + 8) + N;   // matrix with padded rows, then the vector
    static constexpr int RES_WARPS = 2;
    static constexpr int SM_WORK = STAGES * STAGE_FLOATS + 2 * N;
    static constexpr int RES_SLOTS = 3;                // tile aggregates a resolver CTA stages, shared by its resolving warps
    static constexpr int SM_RES = RES_SLOTS * AGG + RES_WARPS * N;
    static constexpr int SM_FLOATS = SM_WORK > SM_RES ? SM_WORK : SM_RES;
    static constexpr size_t SMEM = SM_FLOATS * sizeof(float) + 128;
    static constexpr int MAX_SEQ_PER_WARP = 8;
};

template <int K> __device__ __forceinline__ void cp_async_wait() { asm volatile("cp.async.wait_group %0;" ::"n"(K) : "memory"); }

// Resolver for n = 64: lane i holds components i and i + 32 of the running state.  An aggregate is 16.6 KB: it is
// fetched by asynchronous copies, all of it in flight at once, into one of the warp's tile slots; a warp that serves
// ONE sequence requests the following tiles (as many as it has slots) while it walks the current one, so the round
// trips stay off the serial walk.  The resolver CTA's `slots` tile slots are shared by its w.res_warps resolving warps
// (small batches: one warp with all the slots).
__device__ __forceinline__ float2 resolver64_walk(const float *stage, float *ysm, float y0v, float y1v, int lane)
{
    constexpr int N = 64, NN = N * N;
    ysm[lane] = y0v; ysm[32 + lane] = y1v;
    __syncwarp();
    // rows lane and lane + 32 and the state as 16-byte pieces, each lane starting at a different piece (the eight lanes
    // of a 128-bit access phase then hit distinct banks): a third of the instructions of the element-wise loop
    const float4 *r0 = reinterpret_cast<const float4 *>(stage + lane * N), *r1 = reinterpret_cast<const float4 *>(stage + (32 + lane) * N);
    const float4 *yb = reinterpret_cast<const float4 *>(ysm);
    float a0 = stage[NN + lane], a1 = stage[NN + 32 + lane], b0 = 0.0f, b1 = 0.0f, c0 = 0.0f, c1 = 0.0f, d0 = 0.0f, d1 = 0.0f;
#pragma unroll
    for (int k = 0; k < N / 4; ++k) {
        const int kk = k ^ (lane & 7);
        const float4 yv = yb[kk], u = r0[kk], v = r1[kk];
        a0 = fmaf(u.x, yv.x, a0); b0 = fmaf(u.y, yv.y, b0); c0 = fmaf(u.z, yv.z, c0); d0 = fmaf(u.w, yv.w, d0);
        a1 = fmaf(v.x, yv.x, a1); b1 = fmaf(v.y, yv.y, b1); c1 = fmaf(v.z, yv.z, c1); d1 = fmaf(v.w, yv.w, d1);
    }
    a0 = (a0 + b0) + (c0 + d0);
    a1 = (a1 + b1) + (c1 + d1);
    __syncwarp();
    return make_float2(a0, a1);
}

__device__ void resolver64(const ScanArgs &a, const OnePassWs &w, float *stage_all, int slots, int rw, int nrw, int lane)
{
    if (a.no_resolve) return;     // (wait-expiry test: nobody publishes entering states)
    using C = Cta64;
    constexpr int N = C::N, AGG = C::AGG;
    const int wib = threadIdx.x >> 5;                              // resolving warp of this CTA
    const int RING = max(1, min(4, slots / w.res_warps));          // this warp's tile slots
    float *stage = stage_all + (size_t)wib * RING * AGG;
    float *ysm = stage_all + (size_t)slots * AGG + wib * N;
    auto fetch = [&](float *dst, const float *src) {
        for (int i = lane; i < AGG / 4; i += 32) cp_async16(dst + 4 * i, src + 4 * i);
        cp_async_commit();
    };
    unsigned spins = 0;
    if (rw + nrw >= a.B) {
        // ---- one sequence: tile i in slot i % RING, one fetch group per tile, up to RING in flight
        const int s = rw;
        if (s >= a.B) return;
        const unsigned *flags = w.flags + (size_t)s * w.nch;
        const float *aggs = w.aggs + (size_t)s * w.nch * AGG;
        unsigned long long *starts = w.starts + (size_t)s * w.nch * N;
        float y0v = 0.0f, y1v = 0.0f;
        if (a.y0) { y0v = a.y0[(size_t)s * N + lane]; y1v = a.y0[(size_t)s * N + 32 + lane]; }
        int c = 0, f = 0;                      // next tile to walk, next tile to fetch
        unsigned fl = (lane < w.nch) ? ld_acquire_u32(flags + lane) : 0u;      // flags of tiles f + lane
        while (c < w.nch) {
            bool progressed = false;
            if (f - c < RING && f < w.nch) {
                const unsigned m = __ballot_sync(0xffffffffu, fl >= 1u);
                __syncwarp();      // orders every lane's aggregate copies below after the acquiring lanes' flag loads
                int r = (m == 0xffffffffu) ? 32 : (__ffs(~m) - 1);
                r = min(r, RING - (f - c));
                for (int i = 0; i < r; ++i) fetch(stage + (size_t)((f + i) % RING) * AGG, aggs + (size_t)(f + i) * AGG);
                if (r > 0) progressed = true;
                f += r;
                fl = (f + lane < w.nch) ? ld_acquire_u32(flags + f + lane) : 0u;
            }
            if (f > c) {
                const int ng = f - c;          // groups in flight, oldest first
                if (ng == 1) cp_async_wait<0>(); else if (ng == 2) cp_async_wait<1>(); else if (ng == 3) cp_async_wait<2>(); else cp_async_wait<3>();
                __syncwarp();
                st_relaxed_u64(starts + (size_t)c * N + lane, LL_FLAG | (unsigned long long)__float_as_uint(y0v));
                st_relaxed_u64(starts + (size_t)c * N + 32 + lane, LL_FLAG | (unsigned long long)__float_as_uint(y1v));
                const float2 yn = resolver64_walk(stage + (size_t)(c % RING) * AGG, ysm, y0v, y1v, lane);
                y0v = yn.x; y1v = yn.y;
                if (lane == 0) w.flags[(size_t)s * w.nch + c] = 0u;     // consumed: cleared for the next launch
                ++c;
                progressed = true;
            }
            if (progressed) spins = 0;
            else if (!keep_spinning(a, spins)) { cp_async_wait<0>(); return; }
        }
        return;
    }
    // ---- several sequences per warp: one tile per visit
    int nseq = 0;
    int pos[C::MAX_SEQ_PER_WARP];
    float ya[C::MAX_SEQ_PER_WARP], yb[C::MAX_SEQ_PER_WARP];
    unsigned fnext[C::MAX_SEQ_PER_WARP];
#pragma unroll
    for (int k = 0; k < C::MAX_SEQ_PER_WARP; ++k) {
        pos[k] = 0; ya[k] = 0.0f; yb[k] = 0.0f; fnext[k] = 0u;
        const int s = rw + k * nrw;
        if (s < a.B) {
            nseq = k + 1;
            if (a.y0) { ya[k] = a.y0[(size_t)s * N + lane]; yb[k] = a.y0[(size_t)s * N + 32 + lane]; }
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
            const int cnt = (m == 0xffffffffu) ? 32 : (__ffs(~m) - 1);
            if (cnt == 0) {
                fnext[k] = (c0 + lane < w.nch) ? ld_acquire_u32(flags + c0 + lane) : 0u;
                continue;
            }
            progressed = true;
            unsigned long long *out = w.starts + ((size_t)s * w.nch + c0) * N;
            float y0v = ya[k], y1v = yb[k];
            for (int q = 0; q < cnt; ++q) {
                st_relaxed_u64(out + q * N + lane, LL_FLAG | (unsigned long long)__float_as_uint(y0v));
                st_relaxed_u64(out + q * N + 32 + lane, LL_FLAG | (unsigned long long)__float_as_uint(y1v));
                fetch(stage, w.aggs + ((size_t)s * w.nch + c0 + q) * AGG);
                cp_async_wait<0>();
                __syncwarp();
                const float2 yn = resolver64_walk(stage, ysm, y0v, y1v, lane);
                y0v = yn.x; y1v = yn.y;
            }
            ya[k] = y0v; yb[k] = y1v;
            if (lane < cnt) w.flags[(size_t)s * w.nch + c0 + lane] = 0u;   // consumed: cleared for the next launch
            pos[k] = c0 + cnt;
            if (pos[k] >= w.nch) --remaining;
            else fnext[k] = (pos[k] + lane < w.nch) ? ld_acquire_u32(flags + pos[k] + lane) : 0u;
        }
        if (progressed) spins = 0;
        else if (!keep_spinning(a, spins)) return;
    }
}

// X <- X * M for the warp's 32 rows; B operands read from the padded stage
template <bool REV>
__device__ __forceinline__ void chain_step64(float (&acc)[2][8][4], const float *Ms, int g, int t)
{
    constexpr int RS = RingRow<64, REV>::RS;
    const float *base = REV ? Ms + (2 * t) * RS + g : Ms + g * RS + 2 * t;
    float nacc[2][8][4];
#pragma unroll
    for (int mm = 0; mm < 2; ++mm)
#pragma unroll
        for (int nn = 0; nn < 8; ++nn)
#pragma unroll
            for (int i = 0; i < 4; ++i) nacc[mm][nn][i] = 0.0f;
#pragma unroll
    for (int kk = 0; kk < 8; ++kk) {
        unsigned ah[2][4], al[2][4];
#pragma unroll
        for (int mm = 0; mm < 2; ++mm) {
            split_tf32(acc[mm][kk][0], ah[mm][0], al[mm][0]);
            split_tf32(acc[mm][kk][2], ah[mm][1], al[mm][1]);
            split_tf32(acc[mm][kk][1], ah[mm][2], al[mm][2]);
            split_tf32(acc[mm][kk][3], ah[mm][3], al[mm][3]);
        }
#pragma unroll
        for (int nn = 0; nn < 8; ++nn) {
            float j0, j1;       // M[8kk+2t][8nn+g], M[8kk+2t+1][8nn+g]
            if (!REV) {
                const float2 f = *reinterpret_cast<const float2 *>(base + 8 * nn * RS + 8 * kk);
                j0 = f.x; j1 = f.y;
            } else {
                j0 = base[8 * kk * RS + 8 * nn];
                j1 = base[8 * kk * RS + RS + 8 * nn];
            }
            unsigned bh[2], bl[2];
            split_tf32(j0, bh[0], bl[0]);
            split_tf32(j1, bh[1], bl[1]);
#pragma unroll
            for (int mm = 0; mm < 2; ++mm) {
                mma_tf32(nacc[mm][nn], al[mm], bh, nacc[mm][nn]);
                mma_tf32(nacc[mm][nn], ah[mm], bl, nacc[mm][nn]);
                mma_tf32(nacc[mm][nn], ah[mm], bh, nacc[mm][nn]);
            }
        }
    }
#pragma unroll
    for (int mm = 0; mm < 2; ++mm)
#pragma unroll
        for (int nn = 0; nn < 8; ++nn)
#pragma unroll
            for (int i = 0; i < 4; ++i) acc[mm][nn][i] = nacc[mm][nn][i];
}

// component `i` of  M^T-form product + vector:  forward  sum_c J[i][c] y[c] + b[i],
// reverse  sum_k J[k][i] y[k] + b[i]
template <bool REV>
__device__ __forceinline__ float matvec64(const float *Ms, const float *ycur, int i)
{
    constexpr int RS = RingRow<64, REV>::RS;
    float s0 = 0.0f, s1 = 0.0f, s2 = 0.0f, s3 = 0.0f;
    if (!REV) {
        const int flip = (i >> 2) & 1;             // rows 4..7 of a quarter-warp start on the odd pieces
        const float *row = Ms + i * RS;
#pragma unroll
        for (int k = 0; k < 16; ++k) {
            const int ch = k ^ flip;
            const float4 jv = *reinterpret_cast<const float4 *>(row + (ch << 2));
            const float4 yv = *reinterpret_cast<const float4 *>(ycur + (ch << 2));
            s0 = fmaf(jv.x, yv.x, s0); s1 = fmaf(jv.y, yv.y, s1);
            s2 = fmaf(jv.z, yv.z, s2); s3 = fmaf(jv.w, yv.w, s3);
        }
    } else {
        const float *col = Ms + i;
#pragma unroll
        for (int k4 = 0; k4 < 16; ++k4) {
            const float4 yv = *reinterpret_cast<const float4 *>(ycur + 4 * k4);
            s0 = fmaf(col[(4 * k4) * RS], yv.x, s0);
            s1 = fmaf(col[(4 * k4 + 1) * RS], yv.y, s1);
            s2 = fmaf(col[(4 * k4 + 2) * RS], yv.z, s2);
            s3 = fmaf(col[(4 * k4 + 3) * RS], yv.w, s3);
        }
    }
    return ((s0 + s1) + (s2 + s3)) + Ms[64 * RS + i];
}

template <bool REV>
__global__ void __launch_bounds__(Cta64::THREADS) scan_cta64_kernel(ScanArgs a, OnePassWs w)
{
    using C = Cta64;
    constexpr int N = C::N, NN = C::NN, AGG = C::AGG, Q = C::Q, S = C::STAGES, RS = RingRow<64, REV>::RS;
    pdl_prologue();
    if (loop_ended(a.st)) return;

    extern __shared__ __align__(16) float smem_raw[];
    float *sm = (float *)(((uintptr_t)smem_raw + 127) & ~(uintptr_t)127);
    float *ring = sm;                              // S x (padded matrix, vector)
    float *ybuf = ring + S * C::STAGE_FLOATS;      // 2 x N: running state of the mat-vec chain
    __shared__ int s_kind, s_seq, s_c, s_abort, s_role;

    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const int g = lane >> 2, t = lane & 3;
    const int T = a.T;

    if (tid == 0) {
        s_abort = 0;
        s_role = (int)atomicAdd(&a.st->role_counter, 1u);
    }
    __syncthreads();
    if (s_role < w.resolvers) {
        if (warp < w.res_warps) resolver64(a, w, sm, C::RES_SLOTS, s_role * w.res_warps + warp, w.resolvers * w.res_warps, lane);
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
            int kind = -1, seq = -1, c = -1;
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
                    const int slot = (q_head + q_cnt) % Q;
                    q_seq[slot] = seq; q_c[slot] = c; ++q_cnt;
                } else {
                    exhausted = true;
                    want_b = q_cnt > 0;
                }
            }
            if (want_b) {
                kind = 1; seq = q_seq[q_head]; c = q_c[q_head];
                q_head = (q_head + 1) % Q; --q_cnt;
            }
            s_kind = kind; s_seq = seq; s_c = c;
        }
        __syncthreads();
        if (s_kind < 0 || s_abort) break;
        const int kind = s_kind, seq = s_seq, c = s_c;
        const int s0 = c * C::L;
        const int cnt = min(C::L, T - s0);
        const size_t tile_index = (size_t)seq * w.nch + c;
        const float *Jseq = a.J + (size_t)seq * T * NN;
        const float *bseq = a.b + (size_t)seq * T * N;

        // stage of scan position s: forward J[s]; reverse J[T-s] (identity at s = 0); vector at t(s)
        auto issue_stage = [&](int q) {
            if (q < cnt) {
                const int s = s0 + q;
                float *dst = ring + (q % S) * C::STAGE_FLOATS;
                if (REV && s == 0) {
                    for (int j = tid; j < NN / 4; j += C::THREADS) {
                        const int row = j >> 4, ch = j & 15;
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
                    const float *src = REV ? Jseq + (size_t)(T - s) * NN : Jseq + (size_t)s * NN;
#pragma unroll
                    for (int u = 0; u < NN / 4 / C::THREADS; ++u) {
                        const int j = tid + u * C::THREADS;
                        cp_async16(dst + (j >> 4) * RS + 4 * (j & 15), src + 4 * j);
                    }
                }
                const size_t tt = REV ? (size_t)(T - 1 - s) : (size_t)s;
                if (tid < N / 4) cp_async16(dst + N * RS + 4 * tid, bseq + tt * N + 4 * tid);
            }
            cp_async_commit();
        };

        if (kind == 0) {
            // ---------------------------------------------- A item
            float acc[2][8][4];
#pragma unroll
            for (int mm = 0; mm < 2; ++mm)
#pragma unroll
                for (int nn = 0; nn < 8; ++nn) {
                    const int r = 32 * warp + 16 * mm + g, cc = 8 * nn + 2 * t;
                    acc[mm][nn][0] = (r == cc) ? 1.0f : 0.0f;
                    acc[mm][nn][1] = (r == cc + 1) ? 1.0f : 0.0f;
                    acc[mm][nn][2] = (r + 8 == cc) ? 1.0f : 0.0f;
                    acc[mm][nn][3] = (r + 8 == cc + 1) ? 1.0f : 0.0f;
                }
            ybuf[tid] = 0.0f;
#pragma unroll
            for (int q = 0; q < S - 1; ++q) issue_stage(q);
#pragma unroll 1
            for (int q = 0; q < cnt; ++q) {
                cp_async_wait<S - 2>();
                __syncthreads();
                issue_stage(q + S - 1);
                const float *Ms = ring + (q % S) * C::STAGE_FLOATS;
                chain_step64<REV>(acc, Ms, g, t);
                ybuf[((q + 1) & 1) * N + tid] = matvec64<REV>(Ms, ybuf + (q & 1) * N, tid);
            }
            cp_async_wait<0>();
            __syncthreads();
            // X = P^T in fragments  ->  P row-major, then beta
            float *dst = w.aggs + tile_index * AGG;
#pragma unroll
            for (int mm = 0; mm < 2; ++mm)
#pragma unroll
                for (int nn = 0; nn < 8; ++nn) {
                    const int r = 32 * warp + 16 * mm + g, cc = 8 * nn + 2 * t;
                    dst[cc * N + r] = acc[mm][nn][0];
                    dst[(cc + 1) * N + r] = acc[mm][nn][1];
                    dst[cc * N + r + 8] = acc[mm][nn][2];
                    dst[(cc + 1) * N + r + 8] = acc[mm][nn][3];
                }
            dst[NN + tid] = ybuf[(cnt & 1) * N + tid];
            __threadfence();
            __syncthreads();
            if (tid == 0) st_release_u32(w.flags + tile_index, 1u);
            continue;
        }

        // -------------------------------------------------- B item
#pragma unroll
        for (int q = 0; q < S - 1; ++q) issue_stage(q);
        {
            const unsigned long long *src = w.starts + tile_index * N;
            unsigned spins = 0;
            bool ok = true;
            for (;;) {
                const unsigned long long v = ld_relaxed_u64(src + tid);
                if (v != 0ull) {
                    ybuf[tid] = __uint_as_float((unsigned)(v & 0xffffffffull));
                    st_relaxed_u64(w.starts + tile_index * N + tid, 0ull);      // consumed: cleared for the next launch
                    break;
                }
                if (!keep_spinning(a, spins)) { ok = false; break; }
            }
            if (!ok) s_abort = 1;
        }
#pragma unroll 1
        for (int q = 0; q < cnt; ++q) {
            cp_async_wait<S - 2>();
            __syncthreads();
            if (s_abort) break;
            issue_stage(q + S - 1);
            const float *Ms = ring + (q % S) * C::STAGE_FLOATS;
            const float yn = matvec64<REV>(Ms, ybuf + (q & 1) * N, tid);
            ybuf[((q + 1) & 1) * N + tid] = yn;
            const int s = s0 + q;
            const size_t vb = ((size_t)seq * T + (REV ? (size_t)(T - 1 - s) : (size_t)s)) * N + tid;
            if (a.yold) mb = max(mb, absdiff_bits(yn, __ldg(a.yold + vb)));
            a.y[vb] = yn;
        }
        cp_async_wait<0>();
        if (s_abort) break;
    }
    cp_async_wait<0>();
    if (a.yold) {
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) mb = max(mb, __shfl_xor_sync(0xffffffffu, mb, o));
        if (lane == 0 && mb) { atomicMax(&a.st->err_bits, mb); __threadfence(); }
    }
    __syncthreads();
    if (tid == 0) scan_epilogue(a.st);
}

}  // namespace deer
