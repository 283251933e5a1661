// Single-pass scan for n = 8 with one WARP per chain and the chain product on tensor cores.
//
// Global protocol as in scan_onepass.cuh: a tile (8 chains x SW positions) gets an A item (fold
// into the tile aggregate, publish) and later a B item (replay from the entering state that a
// resolver warp published, write y); the tile's second read is served by L2.  Inside a CTA:
//   * each of the 8 warps owns one chain of SW consecutive positions and streams its J_t straight
//     from global memory: one coalesced 256-byte load per position (lane l reads floats 2l, 2l+1),
//     software-prefetched a group of positions ahead in registers.  No shared-memory staging.
//   * A item: the running product is kept TRANSPOSED, X = P^T with beta^T as a ninth row, in the
//     accumulator fragment of mma.sync.m16n8k8 (TF32 inputs, fp32 accumulate):
//         [X; beta^T] <- [X; beta^T] * J_t^T + [0; b_t^T].
//     The accumulator fragment (row g, columns 2t, 2t+1 in lane 4g+t) is reused as the next A
//     operand without any shuffle by renaming the contraction index (k-slot t <-> column 2t,
//     k-slot t+4 <-> column 2t+1); the B operand then is exactly the lane's 8-byte piece of J_t.
//     Each product is issued as three MMAs on hi/lo TF32 splits (hi*hi + hi*lo + lo*hi), which
//     keeps fp32-level accuracy.
//   * B item: y <- J_t y + b_t as a shuffle mat-vec from the same 8-byte pieces.
//   * The 8 warp aggregates of a tile are combined through shared memory (once per tile).
// Reverse scans use J[t+1]^T: only the addressing of the lane's piece changes.
#pragma once
#include "scan_onepass.cuh"

namespace deer {

struct Warp8 {
    static constexpr int N = 8, NN = 64, AGG = 72;
    static constexpr int WARPS = 8, THREADS = 256;
    static constexpr int SW_MIN = 32, SW_MAX = 256;    // positions per warp chain (chosen per problem size)
    static constexpr int GRP = 8;                      // positions loaded ahead per group
    static constexpr int Q = 2;                        // pending tiles per CTA
    static constexpr int RES_WARPS = 4;                // warps of a resolver CTA that resolve
    static constexpr int PEND = WARPS * AGG;           // warp aggregates kept for the B item
    static constexpr int SM_WORK = Q * PEND + WARPS * N + N + 16;
    static constexpr int SM_RES = RES_WARPS * 32 * AGG;
    static constexpr int SM_FLOATS = SM_WORK > SM_RES ? SM_WORK : SM_RES;
    static constexpr size_t SMEM = SM_FLOATS * sizeof(float) + 128;
    static_assert(SW_MIN % GRP == 0, "chains are processed in whole groups");
    // Longer chains mean fewer tiles for the resolvers to walk (their per-tile cost is what bounds
    // the scan at large T), shorter ones more tiles to spread over the SMs: take the longest
    // chain that still leaves about 1.5 tiles per resident CTA (measured optimum for B = 16,
    // T = 3e3 ... 1e6).
    static int chain_len(int B, int T, int resident_ctas)
    {
        auto tiles = [&](int sw) { return (long long)B * ((T + WARPS * sw - 1) / (WARPS * sw)); };
        int sw = SW_MAX;
        while (sw > SW_MIN && tiles(sw) < 3LL * resident_ctas / 2) sw >>= 1;
        // a nearly empty second wave costs a whole extra item per CTA: if chains at most twice as
        // long bring every tile into the first wave (a few CTAs are resolvers), take them
        const long long workers = resident_ctas - 8;
        if (tiles(sw) > workers)
            for (int s2 = sw + GRP; s2 <= 2 * sw && s2 <= SW_MAX; s2 += GRP)
                if (tiles(s2) <= workers) { sw = s2; break; }
        return sw;
    }
};

__device__ __forceinline__ void prefetch_l1(const void *p) { asm volatile("prefetch.global.L1 [%0];" ::"l"(p)); }

// d = a * b + c   (m16n8k8, A row-major 16x8, B 8x8, TF32 inputs, fp32 accumulate)
__device__ __forceinline__ void mma_tf32(float (&d)[4], const unsigned (&a)[4], const unsigned (&b)[2], const float (&c)[4])
{
    asm volatile("mma.sync.aligned.m16n8k8.row.col.f32.tf32.tf32.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%10,%11,%12,%13};"
                 : "=f"(d[0]), "=f"(d[1]), "=f"(d[2]), "=f"(d[3])
                 : "r"(a[0]), "r"(a[1]), "r"(a[2]), "r"(a[3]), "r"(b[0]), "r"(b[1]),
                   "f"(c[0]), "f"(c[1]), "f"(c[2]), "f"(c[3]));
}

// hi / lo TF32 split by truncation: hi keeps the top 10 mantissa bits, lo the next 10 of the exact
// remainder, so hi*hi + hi*lo + lo*hi carries about 21 mantissa bits of every product.  The tensor
// core reads only the upper 19 bits of a TF32 operand register, so neither half needs masking:
// hi is x itself, lo is x minus its truncation (bit-identical to the masked form on sm_100a).
__device__ __forceinline__ void split_tf32(float x, unsigned &hi, unsigned &lo)
{
    hi = __float_as_uint(x);
    lo = __float_as_uint(x - __uint_as_float(hi & 0xffffe000u));
}

// one step of the transposed chain on the accumulator fragment:
//   [X; beta^T] <- [X; beta^T] * M + [0; (bx, by)]   with the lane's piece (j0, j1) of M
__device__ __forceinline__ void chain_step(float (&acc)[4], float j0, float j1, float bx, float by)
{
    unsigned ah[4], al[4], bh[2], bl[2];
    split_tf32(acc[0], ah[0], al[0]);      // a0 <- c0
    split_tf32(acc[2], ah[1], al[1]);      // a1 <- c2
    split_tf32(acc[1], ah[2], al[2]);      // a2 <- c1
    split_tf32(acc[3], ah[3], al[3]);      // a3 <- c3
    split_tf32(j0, bh[0], bl[0]);
    split_tf32(j1, bh[1], bl[1]);
    // the two small products chain through one accumulator, the large one runs beside them (the next
    // step waits for two MMA latencies and four adds; measured best of: all three independent, this, all chained)
    const float z[4] = {0.0f, 0.0f, 0.0f, 0.0f};
    float d0[4] = {0.0f, 0.0f, bx, by}, d1[4];
    mma_tf32(d1, al, bh, z);
    mma_tf32(d0, ah, bh, d0);
    mma_tf32(d1, ah, bl, d1);
#pragma unroll
    for (int i = 0; i < 4; ++i) acc[i] = d0[i] + d1[i];
}

// Resolver for n = 8 (see resolver_loop of scan_onepass.cuh).  The walk Y <- A Y + beta is the critical
// path of a latency-bound scan, so a step is kept short: lane (r, p) = (lane / 4, lane % 4) holds
// Y[2p], Y[2p+1]; one step is two FMAs on the lane's 8-byte piece of row r, two xor-shuffles, the add
// of beta[r] and two shuffles that hand the new pair to every lane (about a dozen instructions).
__device__ void resolver_loop8(const ScanArgs &a, const OnePassWs &w, float *stage_all, int rw, int nrw, int lane)
{
    if (a.no_resolve) return;     // (wait-expiry test: nobody publishes entering states)
    constexpr int N = 8, NN = 64, AGG = 72, MAXS = OnePass<8>::MAX_SEQ_PER_WARP;
    float *stage = stage_all + (threadIdx.x >> 5) * 32 * AGG;
    const int r = lane >> 2, p = lane & 3;
    int nseq = 0;
    int pos[MAXS];
    float ya[MAXS], yb[MAXS];
    unsigned fnext[MAXS];
#pragma unroll
    for (int k = 0; k < MAXS; ++k) {
        pos[k] = 0; ya[k] = 0.0f; yb[k] = 0.0f; fnext[k] = 0u;
        const int s = rw + k * nrw;
        if (s < a.B) {
            nseq = k + 1;
            if (a.y0) { ya[k] = a.y0[(size_t)s * N + 2 * p]; yb[k] = a.y0[(size_t)s * N + 2 * p + 1]; }
            if (lane < w.nch) fnext[k] = ld_acquire_u32(w.flags + (size_t)s * w.nch + lane);
        }
    }
    int remaining = nseq;
    unsigned spins = 0;
    while (remaining > 0) {
        bool progressed = false;
#pragma unroll
        for (int k = 0; k < MAXS; ++k) {
            if (k >= nseq) break;
            const int c0 = pos[k];
            if (c0 >= w.nch) continue;
            const int s = rw + k * nrw;
            const unsigned *flags = w.flags + (size_t)s * w.nch;
            const unsigned m = __ballot_sync(0xffffffffu, fnext[k] >= 1u);
            __syncwarp();      // orders every lane's aggregate loads below after the acquiring lanes' flag loads
            const int cnt = (m == 0xffffffffu) ? 32 : (__ffs(~m) - 1);
            {
                const int j = c0 + cnt + lane;
                fnext[k] = (j < w.nch) ? ld_acquire_u32(flags + j) : 0u;
            }
            if (cnt == 0) continue;
            progressed = true;
            const float *src = w.aggs + ((size_t)s * w.nch + c0) * AGG;
            {   // the whole batch in flight at once: asynchronous 16-byte copies straight into the stage
                const int total4 = cnt * AGG / 4;
                for (int i = lane; i < total4; i += 32) cp_async16(stage + 4 * i, src + 4 * i);
                cp_async_commit();
                cp_async_wait_0();
            }
            __syncwarp();
            unsigned long long *out = w.starts + ((size_t)s * w.nch + c0) * N;
            float y0v = ya[k], y1v = yb[k];
#pragma unroll 2
            for (int q = 0; q < cnt; ++q) {
                if (r == 0) {
                    st_relaxed_u64(out + q * N + 2 * p, LL_FLAG | (unsigned long long)__float_as_uint(y0v));
                    st_relaxed_u64(out + q * N + 2 * p + 1, LL_FLAG | (unsigned long long)__float_as_uint(y1v));
                }
                const float *ag = stage + q * AGG;
                const float2 a2 = *reinterpret_cast<const float2 *>(ag + r * N + 2 * p);
                float part = fmaf(a2.x, y0v, a2.y * y1v);
                part += __shfl_xor_sync(0xffffffffu, part, 1);
                part += __shfl_xor_sync(0xffffffffu, part, 2);
                const float yn = part + ag[NN + r];
                y0v = __shfl_sync(0xffffffffu, yn, 8 * p);
                y1v = __shfl_sync(0xffffffffu, yn, 8 * p + 4);
            }
            ya[k] = y0v; yb[k] = y1v;
            __syncwarp();
            if (lane < cnt) w.flags[(size_t)s * w.nch + c0 + lane] = 0u;   // consumed: cleared for the next launch
            pos[k] = c0 + cnt;
            if (pos[k] >= w.nch) --remaining;
        }
        if (progressed) spins = 0;
        else if (!keep_spinning(a, spins)) return;
    }
}

template <bool REV>
__global__ void __launch_bounds__(Warp8::THREADS, 4) scan_warp8_kernel(ScanArgs a, OnePassWs w)
{
    using C = Warp8;
    constexpr int N = C::N, NN = C::NN, AGG = C::AGG, WARPS = C::WARPS, GRP = C::GRP, Q = C::Q;
    pdl_prologue();
    const int SW = w.sw, L = WARPS * SW;

    extern __shared__ __align__(16) float smem_raw[];
    float *sm = (float *)(((uintptr_t)smem_raw + 127) & ~(uintptr_t)127);
    float *pend = sm;                          // Q x warp aggregates (A row-major, then beta)
    float *wstart = pend + Q * C::PEND;        // WARPS x N states entering each warp chain
    float *ystart = wstart + WARPS * N;
    __shared__ int s_kind, s_seq, s_c, s_slot, s_abort, s_role, s_done;

    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const int g = lane >> 2, t = lane & 3;     // fragment coordinates
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
        if (warp < C::RES_WARPS)
            resolver_loop8(a, w, sm, s_role * C::RES_WARPS + warp, w.resolvers * C::RES_WARPS, lane);
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
    // tile ids come from the same counter as the role tickets (ticket - resolvers): a worker's ticket
    // is its first tile id (no second atomic before the first tile), and ids are still handed out in
    // order to running CTAs only
    bool first_claim = true;

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
        float *wagg = pend + s_slot * C::PEND;
        const int s0 = c * L;                                  // first scan position of the tile
        const int Lt = min(L, T - s0);
        const int p0 = warp * SW;                              // first scan offset of this warp's chain
        const int cnt = min(SW, max(0, Lt - p0));
        const size_t tile_index = (size_t)seq * w.nch + c;
        const float *Jseq = a.J + (size_t)seq * T * NN;
        const float *bseq = a.b + (size_t)seq * T * N;

        const int sbase = s0 + p0;                             // scan position of the chain's first element
        // per-lane pointers at the chain's first position; the piece advances by a constant per position
        //   forward: float2 #lane of J[s]            (+32 float2 per position), b[s] pairs (+4 float2)
        //   reverse: J[T-s] entries (2t,g),(2t+1,g)  (-64 floats per position), b[T-1-s] (-4 float2)
        const float2 *jp2 = reinterpret_cast<const float2 *>(Jseq + (size_t)sbase * NN) + lane;
        const float *jpr = Jseq + (size_t)(T - sbase) * NN + (2 * t) * N + g;
        const size_t tb = REV ? (size_t)(T - 1 - sbase) : (size_t)sbase;
        auto piece = [&](int q, float &j0, float &j1) {
            if (!REV) { const float2 f = __ldg(jp2 + q * 32); j0 = f.x; j1 = f.y; }
            else if (sbase + q == 0) { j0 = (g == 2 * t) ? 1.0f : 0.0f; j1 = (g == 2 * t + 1) ? 1.0f : 0.0f; }
            else { j0 = __ldg(jpr - q * NN); j1 = __ldg(jpr - q * NN + N); }
        };

        if (kind == 0) {
            // ---------------------------------------------- A item: [X; beta^T] in the accumulator fragment
            float acc[4] = {(g == 2 * t) ? 1.0f : 0.0f, (g == 2 * t + 1) ? 1.0f : 0.0f, 0.0f, 0.0f};
            const float2 *bp2 = reinterpret_cast<const float2 *>(bseq + tb * N) + t;
            const float *bch = bseq + tb * N;
            // whole groups: loads with constant offsets from one pointer per group, no per-position tests
            int q0 = 0;
            if (REV && sbase == 0 && cnt > 0) {                 // scan position 0 of the reverse scan: identity
                const float2 f = (g == 0) ? __ldg(bp2) : make_float2(0.0f, 0.0f);
                chain_step(acc, (g == 2 * t) ? 1.0f : 0.0f, (g == 2 * t + 1) ? 1.0f : 0.0f, f.x, f.y);
                q0 = 1;
            }
#pragma unroll 1
            for (; q0 + GRP <= cnt; q0 += GRP) {
                float j0[GRP], j1[GRP], bx[GRP], by[GRP];
                const float2 *jq = jp2 + q0 * 32;
                const float *jr = jpr - q0 * NN;
                const float2 *bq = REV ? bp2 - q0 * 4 : bp2 + q0 * 4;
                if (q0 + 2 * GRP <= cnt) {              // next group towards L1 while this one is used
#pragma unroll
                    for (int u = 0; u < GRP; ++u) {
                        if (!REV) prefetch_l1(jq + (GRP + u) * 32);
                        else { prefetch_l1(jr - (GRP + u) * NN); prefetch_l1(jr - (GRP + u) * NN + N); }
                    }
                    // the next group's b: 256 contiguous bytes, up to three lines
                    if (lane < 3) prefetch_l1(bch + (REV ? -(q0 + 2 * GRP - 1) * N : (q0 + GRP) * N) + min(lane * 32, GRP * N - 1));
                }
#pragma unroll
                for (int u = 0; u < GRP; ++u) {
                    if (!REV) { const float2 f = __ldg(jq + u * 32); j0[u] = f.x; j1[u] = f.y; }
                    else { j0[u] = __ldg(jr - u * NN); j1[u] = __ldg(jr - u * NN + N); }
                    bx[u] = 0.0f; by[u] = 0.0f;
                    if (g == 0) { const float2 f = __ldg(REV ? bq - u * 4 : bq + u * 4); bx[u] = f.x; by[u] = f.y; }
                }
#pragma unroll
                for (int u = 0; u < GRP; ++u) chain_step(acc, j0[u], j1[u], bx[u], by[u]);
            }
#pragma unroll 1
            for (; q0 < cnt; ++q0) {                            // ragged tail
                float j0, j1, bx = 0.0f, by = 0.0f;
                piece(q0, j0, j1);
                if (g == 0) { const float2 f = __ldg(REV ? bp2 - q0 * 4 : bp2 + q0 * 4); bx = f.x; by = f.y; }
                chain_step(acc, j0, j1, bx, by);
            }
            // X[g][2t] = P[2t][g], X[g][2t+1] = P[2t+1][g]; beta in row 8 (lanes with g == 0)
            {
                float *ag = wagg + warp * AGG;
                ag[(2 * t) * N + g] = acc[0];
                ag[(2 * t + 1) * N + g] = acc[1];
                if (g == 0) { ag[NN + 2 * t] = acc[2]; ag[NN + 2 * t + 1] = acc[3]; }
            }
            __syncthreads();
            if (warp == 0) {
                // tile aggregate: the same step with the warp aggregates as "positions" (forward form:
                // piece (g,2t),(g,2t+1) of A_k, beta_k as the additive row)
                float tac[4] = {(g == 2 * t) ? 1.0f : 0.0f, (g == 2 * t + 1) ? 1.0f : 0.0f, 0.0f, 0.0f};
#pragma unroll
                for (int k = 0; k < WARPS; ++k) {
                    float *ak = wagg + k * AGG;
                    const float2 f = *reinterpret_cast<const float2 *>(ak + 2 * lane);
                    float bx = 0.0f, by = 0.0f;
                    if (g == 0) { bx = ak[NN + 2 * t]; by = ak[NN + 2 * t + 1]; }
                    chain_step(tac, f.x, f.y, bx, by);
                    // warp k's aggregate is replaced by the aggregate of warps 0..k: in the B item every
                    // warp then gets the state entering its chain by one mat-vec of its own
                    __syncwarp();
                    ak[(2 * t) * N + g] = tac[0];
                    ak[(2 * t + 1) * N + g] = tac[1];
                    if (g == 0) { ak[NN + 2 * t] = tac[2]; ak[NN + 2 * t + 1] = tac[3]; }
                }
                float *gdst = w.aggs + tile_index * AGG;
                gdst[(2 * t) * N + g] = tac[0];
                gdst[(2 * t + 1) * N + g] = tac[1];
                if (g == 0) { gdst[NN + 2 * t] = tac[2]; gdst[NN + 2 * t + 1] = tac[3]; }
                __threadfence();
                __syncwarp();
                if (lane == 0) st_release_u32(w.flags + tile_index, 1u);
            }
            continue;
        }

        // -------------------------------------------------- B item
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
        if (s_abort) break;
        if (warp == 0) {
            if (lane < N) wstart[lane] = ystart[lane];
            __syncwarp();
        } else {
            matvec_smem<8>(wstart + warp * N, wagg + (warp - 1) * AGG, ystart, lane);
        }
        {
            // lane (g,t) carries y[2t], y[2t+1]; every step: partial sums over k = 2t, 2t+1, reduced over t
            float yk0 = wstart[warp * N + 2 * t], yk1 = wstart[warp * N + 2 * t + 1];
            const float *bpg = bseq + tb * N + g;
            const float *yop = a.yold ? a.yold + ((size_t)seq * T + tb) * N + g : nullptr;
            float *yp = a.y + ((size_t)seq * T + tb) * N + g;
            auto step = [&](float j0, float j1, float bgv, float yov, int off) {
                float part = fmaf(j0, yk0, j1 * yk1);
                part += __shfl_xor_sync(0xffffffffu, part, 1);
                part += __shfl_xor_sync(0xffffffffu, part, 2);
                const float yg = part + bgv;                                    // y_new[g], in all 4 lanes of group g
                yk0 = __shfl_sync(0xffffffffu, yg, 4 * (2 * t));
                yk1 = __shfl_sync(0xffffffffu, yg, 4 * (2 * t + 1));
                if (t == 0) {
                    if (yop) mb = max(mb, absdiff_bits(yg, yov));
                    yp[off] = yg;
                }
            };
            int q0 = 0;
            if (REV && sbase == 0 && cnt > 0) {
                float yov = 0.0f;
                if (yop && t == 0) yov = __ldg(yop);
                step((g == 2 * t) ? 1.0f : 0.0f, (g == 2 * t + 1) ? 1.0f : 0.0f, __ldg(bpg), yov, 0);
                q0 = 1;
            }
            static_assert(GRP % 4 == 0, "lane (g,t) writes positions t, t+4, ... of a group");
#pragma unroll 1
            for (; q0 + GRP <= cnt; q0 += GRP) {
                float j0[GRP], j1[GRP], bg[GRP], yg[GRP];
                const float2 *jq = jp2 + q0 * 32;
                const float *jr = jpr - q0 * NN;
                const int off0 = REV ? -q0 * N : q0 * N;
                if (q0 + 2 * GRP <= cnt) {
#pragma unroll
                    for (int u = 0; u < GRP; ++u) {
                        if (!REV) prefetch_l1(jq + (GRP + u) * 32);
                        else { prefetch_l1(jr - (GRP + u) * NN); prefetch_l1(jr - (GRP + u) * NN + N); }
                    }
                    // the next group's b and y_old: 256 contiguous bytes each, up to three lines
                    const int nx = (REV ? -(q0 + 2 * GRP - 1) * N : (q0 + GRP) * N) + min((lane & 3) * 32, GRP * N - 1);
                    if (lane < 3) prefetch_l1(bpg - g + nx);
                    else if (yop && lane >= 4 && lane < 7) prefetch_l1(yop - g + nx);
                }
                const int offt = off0 + (REV ? -t * N : t * N);               // this lane's first position of the group
                float yo[GRP / 4];
#pragma unroll
                for (int h = 0; h < GRP / 4; ++h) yo[h] = yop ? __ldg(yop + offt + (REV ? -4 * h * N : 4 * h * N)) : 0.0f;
#pragma unroll
                for (int u = 0; u < GRP; ++u) {
                    if (!REV) { const float2 f = __ldg(jq + u * 32); j0[u] = f.x; j1[u] = f.y; }
                    else { j0[u] = __ldg(jr - u * NN); j1[u] = __ldg(jr - u * NN + N); }
                    bg[u] = __ldg(bpg + off0 + (REV ? -u * N : u * N));
                }
#pragma unroll
                for (int u = 0; u < GRP; ++u) {
                    float part = fmaf(j0[u], yk0, j1[u] * yk1);
                    part += __shfl_xor_sync(0xffffffffu, part, 1);
                    part += __shfl_xor_sync(0xffffffffu, part, 2);
                    yg[u] = part + bg[u];                                       // y_new[g], in all 4 lanes of group g
                    yk0 = __shfl_sync(0xffffffffu, yg[u], 4 * (2 * t));
                    yk1 = __shfl_sync(0xffffffffu, yg[u], 4 * (2 * t + 1));
                }
                // lane (g,t) writes component g of positions t, t+4, ...: stores of 128 contiguous bytes
#pragma unroll
                for (int h = 0; h < GRP / 4; ++h) {
                    const float mine = t == 0 ? yg[4 * h] : t == 1 ? yg[4 * h + 1] : t == 2 ? yg[4 * h + 2] : yg[4 * h + 3];
                    if (yop) mb = max(mb, absdiff_bits(mine, yo[h]));
                    yp[offt + (REV ? -4 * h * N : 4 * h * N)] = mine;
                }
            }
#pragma unroll 1
            for (; q0 < cnt; ++q0) {
                float j0, j1, yov = 0.0f;
                const int off = REV ? -q0 * N : q0 * N;
                piece(q0, j0, j1);
                if (yop && t == 0) yov = __ldg(yop + off);
                step(j0, j1, __ldg(bpg + off), yov, off);
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
