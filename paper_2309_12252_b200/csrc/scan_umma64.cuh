// Single-pass scan for n = 64 with the chain product on the 5th-generation tensor cores (tcgen05).
//
// A tile is one chain advanced by a 128-thread CTA.  The running product X = P^T (64 x 64) is the A
// operand of the next step and the accumulator of the current one:
//       D = X * M,   M = J_t^T (forward)  or  J_{t+1} (reverse),
// issued as tcgen05.mma.kind::tf32 with M = 64, N = 64, K = 8: eight K steps, each three times on the
// hi / lo TF32 halves of both operands (lo*hi, hi*lo, hi*hi; fp32-level accuracy), 24 instructions per
// position from one thread, D in tensor memory.  Per position:
//   * the raw matrix (16 KB) arrives through a cp.async ring (rows padded to 68 floats);
//   * all threads rewrite it as the B operand, hi and lo parts, in the canonical K-major
//     SWIZZLE_128B layout (two column halves of [64 rows][128 B], 16-byte pieces XORed with row % 8);
//     the forward direction copies rows, the reverse direction transposes (B must be K-major:
//     B[k][n] is stored at row n, column k);
//   * 64 threads advance the fp32 mat-vec chain for beta from the raw matrix meanwhile;
//   * after the MMAs have been committed to an mbarrier, the four warps read D back with tcgen05.ld
//     (warp w sees rows 16w .. 16w+15 in its lanes 0 .. 15), split it and store hi / lo as the next
//     A operand (same layout).
// The B item (replay from the entering state) is the fp32 mat-vec of scan_cta64.cuh.  Tiles, items,
// resolvers, flags and bounded waits are those of scan_onepass.cuh; every wait on the mbarrier is
// bounded, and the CTA frees its tensor memory on every exit path.
#pragma once
#include "scan_cta64.cuh"

namespace deer {

struct Umma64 {
    static constexpr int N = 64, NN = N * N, AGG = NN + N;
    static constexpr int THREADS = 128;
    static constexpr int L = 64;                       // positions per tile
    static constexpr int Q = 2;                        // pending tiles per CTA
    static constexpr int STAGES = 2;                   // raw ring depth (positions)
    static constexpr int RS = 68;                      // row stride of a raw matrix (floats)
    static constexpr int RAW_FLOATS = N * RS + N;      // raw matrix, then the vector
    static constexpr int OPERAND_BYTES = 16384;        // one 64 x 64 fp32 operand in canonical layout
    static constexpr int RES_WARPS = 4;
    static constexpr int MAX_SEQ_PER_WARP = 8;
    static constexpr size_t SM_WORK = 4 * OPERAND_BYTES + sizeof(float) * (STAGES * RAW_FLOATS + 2 * N);   // reverse; forward:
    static_assert(6 * OPERAND_BYTES + sizeof(float) * 4 * N <= SM_WORK, "the forward layout fits the same allocation");
    static constexpr size_t SM_RES = sizeof(float) * RES_WARPS * (AGG + N);
    static constexpr size_t SMEM = (SM_WORK > SM_RES ? SM_WORK : SM_RES) + 1024;
    static constexpr unsigned TMEM_COLS = 64;
};

// byte offset of element (row, col) of a 64 x 64 fp32 operand in the K-major SWIZZLE_128B layout
__device__ __forceinline__ int umma_off(int row, int col)
{
    return (col >> 5) * 8192 + row * 128 + ((((col & 31) >> 2) ^ (row & 7)) << 4) + ((col & 3) << 2);
}

// shared-memory matrix descriptor (sm_100): start address, leading / stride byte offsets in 16-byte
// units, descriptor version 1, SWIZZLE_128B
__device__ __forceinline__ uint64_t umma_desc(unsigned saddr)
{
    uint64_t d = 0;
    d |= (uint64_t)((saddr >> 4) & 0x3FFF);
    d |= (uint64_t)1 << 16;                 // leading byte offset: unused for swizzled K-major operands
    d |= (uint64_t)(1024 >> 4) << 32;       // stride byte offset: 8 rows x 128 B between row groups
    d |= 1ull << 46;
    d |= 2ull << 61;
    return d;
}

__device__ __forceinline__ void umma_tf32(unsigned tmem_d, uint64_t da, uint64_t db, unsigned idesc, unsigned accumulate)
{
    asm volatile(
        "{\n\t"
        ".reg .pred p;\n\t"
        "setp.ne.b32 p, %4, 0;\n\t"
        "tcgen05.mma.cta_group::1.kind::tf32 [%0], %1, %2, %3, {%5, %6, %7, %8}, p; \n\t"
        "}\n"
        :
        : "r"(tmem_d), "l"(da), "l"(db), "r"(idesc), "r"(accumulate), "r"(0u), "r"(0u), "r"(0u), "r"(0u)
        : "memory");
}

__device__ __forceinline__ void tmem_ld32(unsigned taddr, unsigned (&v)[32])
{
    asm volatile("tcgen05.ld.sync.aligned.32x32b.x32.b32"
                 "{%0, %1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15,"
                 "%16, %17, %18, %19, %20, %21, %22, %23, %24, %25, %26, %27, %28, %29, %30, %31}, [%32];\n"
                 : "=r"(v[0]), "=r"(v[1]), "=r"(v[2]), "=r"(v[3]), "=r"(v[4]), "=r"(v[5]), "=r"(v[6]), "=r"(v[7]),
                   "=r"(v[8]), "=r"(v[9]), "=r"(v[10]), "=r"(v[11]), "=r"(v[12]), "=r"(v[13]), "=r"(v[14]), "=r"(v[15]),
                   "=r"(v[16]), "=r"(v[17]), "=r"(v[18]), "=r"(v[19]), "=r"(v[20]), "=r"(v[21]), "=r"(v[22]), "=r"(v[23]),
                   "=r"(v[24]), "=r"(v[25]), "=r"(v[26]), "=r"(v[27]), "=r"(v[28]), "=r"(v[29]), "=r"(v[30]), "=r"(v[31])
                 : "r"(taddr));
}

__device__ __forceinline__ float tf32_lo(float x) { return x - __uint_as_float(__float_as_uint(x) & 0xffffe000u); }

// component `i` of  M^T-form product + vector from a raw stage (rows of 68 floats: the row reads of
// eight consecutive rows and the column reads fall into distinct banks):
//   forward  sum_c J[i][c] y[c] + b[i],   reverse  sum_k J[k][i] y[k] + b[i]
template <bool REV>
__device__ __forceinline__ float matvec_raw64(const float *Ms, const float *ycur, int i)
{
    constexpr int RS = Umma64::RS;
    float s0 = 0.0f, s1 = 0.0f, s2 = 0.0f, s3 = 0.0f;
    if (!REV) {
        const float *row = Ms + i * RS;
#pragma unroll
        for (int k = 0; k < 16; ++k) {
            const float4 jv = *reinterpret_cast<const float4 *>(row + 4 * k);
            const float4 yv = *reinterpret_cast<const float4 *>(ycur + 4 * k);
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

// forward mat-vec straight from a staged B operand (hi part = the raw matrix in the swizzled layout):
// component i of  sum_c J[i][c] y[c] + b[i]; eight consecutive rows read eight different 16-byte pieces
__device__ __forceinline__ float matvec_swz64(const unsigned char *Bh, const float *bvec, const float *ycur, int i)
{
    float s0 = 0.0f, s1 = 0.0f, s2 = 0.0f, s3 = 0.0f;
    const unsigned char *row = Bh + i * 128;
    const int x = i & 7;
#pragma unroll
    for (int k = 0; k < 16; ++k) {
        const float4 jv = *reinterpret_cast<const float4 *>(row + (k >> 3) * 8192 + (((k & 7) ^ x) << 4));
        const float4 yv = *reinterpret_cast<const float4 *>(ycur + 4 * k);
        s0 = fmaf(jv.x, yv.x, s0); s1 = fmaf(jv.y, yv.y, s1);
        s2 = fmaf(jv.z, yv.z, s2); s3 = fmaf(jv.w, yv.w, s3);
    }
    return ((s0 + s1) + (s2 + s3)) + bvec[i];
}

template <bool REV>
__global__ void __launch_bounds__(Umma64::THREADS) scan_umma64_kernel(ScanArgs a, OnePassWs w)
{
    using C = Umma64;
    constexpr int N = C::N, NN = C::NN, AGG = C::AGG, Q = C::Q, S = C::STAGES, RS = C::RS;
    pdl_prologue();
    if (loop_ended(a.st)) return;

    extern __shared__ __align__(16) unsigned char smem_bytes[];
    unsigned char *sm = (unsigned char *)(((uintptr_t)smem_bytes + 1023) & ~(uintptr_t)1023);
    unsigned char *sAh = sm, *sAl = sm + C::OPERAND_BYTES, *sBh = sm + 2 * C::OPERAND_BYTES, *sBl = sm + 3 * C::OPERAND_BYTES;
    float *ring = reinterpret_cast<float *>(sm + 4 * C::OPERAND_BYTES);     // S x (raw matrix, vector)
    float *ybuf = ring + S * C::RAW_FLOATS;                                  // 2 x N: state of the mat-vec chain
    __shared__ __align__(8) uint64_t s_mbar;
    __shared__ unsigned s_tmem;
    __shared__ int s_kind, s_seq, s_c, s_abort, s_role;

    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const int T = a.T;

    if (tid == 0) {
        s_abort = 0;
        s_role = (int)atomicAdd(&a.st->role_counter, 1u);
    }
    __syncthreads();
    if (s_role < w.resolvers) {
        if (warp < C::RES_WARPS)
            resolver64(a, w, reinterpret_cast<float *>(sm), C::RES_WARPS, s_role * C::RES_WARPS + warp, w.resolvers * C::RES_WARPS, lane);
        __syncthreads();
        if (tid == 0) scan_epilogue(a.st);
        return;
    }
    // worker: tensor memory for the accumulator, one mbarrier for MMA completion
    if (tid == 0) mbar_init(&s_mbar, 1);
    if (warp == 0) {
        asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(&s_tmem)), "r"(C::TMEM_COLS) : "memory");
        asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
    }
    asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
    __syncthreads();
    asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
    const unsigned tmem = s_tmem;
    // instruction descriptor: D fp32, A and B TF32, both K-major, N = 64, M = 64
    constexpr unsigned IDESC = (1u << 4) | (2u << 7) | (2u << 10) | ((64u >> 3) << 17) | ((64u >> 4) << 24);
    unsigned mphase = 0;
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

        // raw stage of scan position s: forward J[s]; reverse J[T-s] (identity at s = 0); vector at t(s)
        auto issue_stage = [&](int q) {
            if (q < cnt) {
                const int s = s0 + q;
                float *dst = ring + (q % S) * C::RAW_FLOATS;
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

        if (kind == 0 && !REV) {
            // ---------------------------------------------- A item, forward: software-pipelined.
            // Shared memory: A hi/lo, two B buffers (hi, lo each), two vectors.  J[s] goes by cp.async
            // straight into the hi part of a B buffer (row-major rows are already K-major); while the
            // MMAs of position q run, the threads make the lo part of position q+1 and advance beta.
            unsigned char *sB[2] = {sm + 2 * C::OPERAND_BYTES, sm + 4 * C::OPERAND_BYTES};      // hi at +0, lo at +16 KB
            float *bvec = reinterpret_cast<float *>(sm + 6 * C::OPERAND_BYTES);                 // 2 x N
            float *yb = bvec + 2 * N;                                                           // 2 x N
            auto stage_fwd = [&](int q) {
                if (q < cnt) {
                    const float *src = Jseq + (size_t)(s0 + q) * NN;
                    unsigned char *dst = sB[q & 1];
#pragma unroll
                    for (int u = 0; u < NN / 4 / C::THREADS; ++u) {
                        const int j = tid + u * C::THREADS;
                        cp_async16(dst + umma_off(j >> 4, 4 * (j & 15)), src + 4 * j);
                    }
                    if (tid < N / 4) cp_async16(bvec + (q & 1) * N + 4 * tid, bseq + (size_t)(s0 + q) * N + 4 * tid);
                }
                cp_async_commit();
            };
            // lo part of the staged matrix and one step of the beta chain (position q)
            auto prepare = [&](int q) {
                unsigned char *B = sB[q & 1];
#pragma unroll
                for (int u = 0; u < NN / 4 / C::THREADS; ++u) {
                    const int off = (tid + u * C::THREADS) * 16;
                    const float4 v = *reinterpret_cast<const float4 *>(B + off);
                    *reinterpret_cast<float4 *>(B + C::OPERAND_BYTES + off) = make_float4(tf32_lo(v.x), tf32_lo(v.y), tf32_lo(v.z), tf32_lo(v.w));
                }
                if (tid < N) yb[((q + 1) & 1) * N + tid] = matvec_swz64(B, bvec + (q & 1) * N, yb + (q & 1) * N, tid);
            };
            for (int j = tid; j < NN / 4; j += C::THREADS) {
                const int row = j >> 4, ch = j & 15;
                float4 v = make_float4(0.f, 0.f, 0.f, 0.f);
                if ((row >> 2) == ch) {
                    if ((row & 3) == 0) v.x = 1.0f;
                    if ((row & 3) == 1) v.y = 1.0f;
                    if ((row & 3) == 2) v.z = 1.0f;
                    if ((row & 3) == 3) v.w = 1.0f;
                }
                *reinterpret_cast<float4 *>(sAh + umma_off(row, 4 * ch)) = v;
                *reinterpret_cast<float4 *>(sAl + umma_off(row, 4 * ch)) = make_float4(0.f, 0.f, 0.f, 0.f);
            }
            if (tid < N) yb[tid] = 0.0f;
            stage_fwd(0);
            stage_fwd(1);
            cp_async_wait<1>();
            __syncthreads();
            prepare(0);
            fence_proxy_async();
            asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
            __syncthreads();
            unsigned xv[64];
#pragma unroll
            for (int i = 0; i < 64; ++i) xv[i] = 0u;
            bool ok = true;
#pragma unroll 1
            for (int q = 0; q < cnt; ++q) {
                if (tid == 0) {
                    asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
                    const unsigned ah = smem_u32(sAh), al = smem_u32(sAl), bh = smem_u32(sB[q & 1]), bl = bh + C::OPERAND_BYTES;
#pragma unroll
                    for (int ks = 0; ks < 8; ++ks) {
                        const unsigned off = (ks >> 2) * 8192 + (ks & 3) * 32;
                        umma_tf32(tmem, umma_desc(al + off), umma_desc(bh + off), IDESC, ks ? 1u : 0u);
                        umma_tf32(tmem, umma_desc(ah + off), umma_desc(bl + off), IDESC, 1u);
                        umma_tf32(tmem, umma_desc(ah + off), umma_desc(bh + off), IDESC, 1u);
                    }
                    asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(smem_u32(&s_mbar)) : "memory");
                }
                // meanwhile: the next position's operand (its matrix was requested one step ago)
                cp_async_wait<0>();
                __syncthreads();
                if (q + 1 < cnt) prepare(q + 1);
                {
                    unsigned spins = 0;
                    while (!mbar_try_wait(&s_mbar, mphase)) {
                        if (++spins > SPIN_LIMIT) { atomicOr(&a.st->flags, FLAG_TIMEOUT); ok = false; break; }
                    }
                    mphase ^= 1u;
                }
                asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
                if (__syncthreads_or(!ok)) { s_abort = 1; break; }
                stage_fwd(q + 2);                  // buffer q & 1 is free: the MMAs of position q are done
                {
                    const unsigned taddr = tmem + ((unsigned)(32 * warp) << 16);
                    unsigned lo32[32], hi32[32];
                    tmem_ld32(taddr, lo32);
                    tmem_ld32(taddr + 32, hi32);
                    asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory");
#pragma unroll
                    for (int i = 0; i < 32; ++i) { xv[i] = lo32[i]; xv[32 + i] = hi32[i]; }
                }
                if (lane < 16 && q + 1 < cnt) {
                    const int row = 16 * warp + lane;
#pragma unroll
                    for (int c4 = 0; c4 < 16; ++c4) {
                        const float4 h = make_float4(__uint_as_float(xv[4 * c4]), __uint_as_float(xv[4 * c4 + 1]),
                                                     __uint_as_float(xv[4 * c4 + 2]), __uint_as_float(xv[4 * c4 + 3]));
                        const int off = umma_off(row, 4 * c4);
                        *reinterpret_cast<float4 *>(sAh + off) = h;
                        *reinterpret_cast<float4 *>(sAl + off) = make_float4(tf32_lo(h.x), tf32_lo(h.y), tf32_lo(h.z), tf32_lo(h.w));
                    }
                }
                fence_proxy_async();
                asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
                __syncthreads();
            }
            cp_async_wait<0>();
            __syncthreads();
            if (s_abort) break;
            float *dst = w.aggs + tile_index * AGG;
            if (lane < 16) {
                const int row = 16 * warp + lane;
#pragma unroll
                for (int cc = 0; cc < 64; ++cc) dst[cc * N + row] = __uint_as_float(xv[cc]);
            }
            if (tid < N) dst[NN + tid] = yb[(cnt & 1) * N + tid];
            __threadfence();
            __syncthreads();
            if (tid == 0) st_release_u32(w.flags + tile_index, 1u);
            continue;
        }
        if (kind == 0) {
            // ---------------------------------------------- A item (reverse: the matrix is transposed while
            // it is rewritten as the B operand, so it goes through a raw stage first)
            // X = I as the first A operand (hi = I, lo = 0); beta chain starts from zero
            for (int j = tid; j < NN / 4; j += C::THREADS) {
                const int row = j >> 4, ch = j & 15;
                float4 v = make_float4(0.f, 0.f, 0.f, 0.f);
                if ((row >> 2) == ch) {
                    if ((row & 3) == 0) v.x = 1.0f;
                    if ((row & 3) == 1) v.y = 1.0f;
                    if ((row & 3) == 2) v.z = 1.0f;
                    if ((row & 3) == 3) v.w = 1.0f;
                }
                *reinterpret_cast<float4 *>(sAh + umma_off(row, 4 * ch)) = v;
                *reinterpret_cast<float4 *>(sAl + umma_off(row, 4 * ch)) = make_float4(0.f, 0.f, 0.f, 0.f);
            }
            if (tid < N) ybuf[tid] = 0.0f;
            issue_stage(0);
            unsigned xv[64];                       // row 16*warp + lane of X (lanes 0..15)
#pragma unroll
            for (int i = 0; i < 64; ++i) xv[i] = (lane < 16 && i == 16 * warp + lane) ? 0x3f800000u : 0u;
            bool ok = true;
#pragma unroll 1
            for (int q = 0; q < cnt; ++q) {
                cp_async_wait<0>();
                __syncthreads();                   // raw stage q landed; the other stage and B operands are free
                issue_stage(q + 1);
                const float *Ms = ring + (q % S) * C::RAW_FLOATS;
                // B operand: hi and lo parts, K-major (row = n, column = k of B[k][n] = M[k][n])
                if (!REV) {
#pragma unroll
                    for (int u = 0; u < NN / 4 / C::THREADS; ++u) {
                        const int j = tid + u * C::THREADS, r = j >> 4, ch = j & 15;
                        const float4 v = *reinterpret_cast<const float4 *>(Ms + r * RS + 4 * ch);
                        const int off = umma_off(r, 4 * ch);
                        *reinterpret_cast<float4 *>(sBh + off) = v;
                        *reinterpret_cast<float4 *>(sBl + off) = make_float4(tf32_lo(v.x), tf32_lo(v.y), tf32_lo(v.z), tf32_lo(v.w));
                    }
                } else {
#pragma unroll
                    for (int u = 0; u < NN / 4 / C::THREADS; ++u) {
                        const int k = lane + 32 * (u & 1), ch = warp * 4 + (u >> 1);
                        const float4 v = *reinterpret_cast<const float4 *>(Ms + k * RS + 4 * ch);
                        const float e[4] = {v.x, v.y, v.z, v.w};
#pragma unroll
                        for (int i = 0; i < 4; ++i) {
                            const int off = umma_off(4 * ch + i, k);
                            *reinterpret_cast<float *>(sBh + off) = e[i];
                            *reinterpret_cast<float *>(sBl + off) = tf32_lo(e[i]);
                        }
                    }
                }
                if (tid < N) ybuf[((q + 1) & 1) * N + tid] = matvec_raw64<REV>(Ms, ybuf + (q & 1) * N, tid);
                fence_proxy_async();
                asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
                __syncthreads();
                if (tid == 0) {
                    asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
                    const unsigned ah = smem_u32(sAh), al = smem_u32(sAl), bh = smem_u32(sBh), bl = smem_u32(sBl);
#pragma unroll
                    for (int ks = 0; ks < 8; ++ks) {
                        const unsigned off = (ks >> 2) * 8192 + (ks & 3) * 32;     // 8 columns = 32 B per K step
                        umma_tf32(tmem, umma_desc(al + off), umma_desc(bh + off), IDESC, ks ? 1u : 0u);
                        umma_tf32(tmem, umma_desc(ah + off), umma_desc(bl + off), IDESC, 1u);
                        umma_tf32(tmem, umma_desc(ah + off), umma_desc(bh + off), IDESC, 1u);
                    }
                    asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(smem_u32(&s_mbar)) : "memory");
                }
                {
                    unsigned spins = 0;
                    while (!mbar_try_wait(&s_mbar, mphase)) {
                        if (++spins > SPIN_LIMIT) { atomicOr(&a.st->flags, FLAG_TIMEOUT); ok = false; break; }
                    }
                    mphase ^= 1u;
                }
                asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
                if (__syncthreads_or(!ok)) { s_abort = 1; break; }      // the whole CTA gives up together
                {
                    const unsigned taddr = tmem + ((unsigned)(32 * warp) << 16);
                    unsigned lo32[32], hi32[32];
                    tmem_ld32(taddr, lo32);
                    tmem_ld32(taddr + 32, hi32);
                    asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory");
#pragma unroll
                    for (int i = 0; i < 32; ++i) { xv[i] = lo32[i]; xv[32 + i] = hi32[i]; }
                }
                if (lane < 16 && q + 1 < cnt) {
                    const int row = 16 * warp + lane;
#pragma unroll
                    for (int c4 = 0; c4 < 16; ++c4) {
                        const float4 h = make_float4(__uint_as_float(xv[4 * c4]), __uint_as_float(xv[4 * c4 + 1]),
                                                     __uint_as_float(xv[4 * c4 + 2]), __uint_as_float(xv[4 * c4 + 3]));
                        const int off = umma_off(row, 4 * c4);
                        *reinterpret_cast<float4 *>(sAh + off) = h;
                        *reinterpret_cast<float4 *>(sAl + off) = make_float4(tf32_lo(h.x), tf32_lo(h.y), tf32_lo(h.z), tf32_lo(h.w));
                    }
                }
            }
            cp_async_wait<0>();
            __syncthreads();
            if (s_abort) break;
            // X = P^T: row r of X is column r of P; then beta
            float *dst = w.aggs + tile_index * AGG;
            if (lane < 16) {
                const int row = 16 * warp + lane;
#pragma unroll
                for (int cc = 0; cc < 64; ++cc) dst[cc * N + row] = __uint_as_float(xv[cc]);
            }
            if (tid < N) dst[NN + tid] = ybuf[(cnt & 1) * N + tid];
            __threadfence();
            __syncthreads();
            if (tid == 0) st_release_u32(w.flags + tile_index, 1u);
            continue;
        }

        // -------------------------------------------------- B item
        issue_stage(0);
        if (tid < N) {
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
            cp_async_wait<0>();
            __syncthreads();
            if (s_abort) break;
            issue_stage(q + 1);
            if (tid < N) {
                const float *Ms = ring + (q % S) * C::RAW_FLOATS;
                const float yn = matvec_raw64<REV>(Ms, ybuf + (q & 1) * N, tid);
                ybuf[((q + 1) & 1) * N + tid] = yn;
                const int s = s0 + q;
                const size_t vb = ((size_t)seq * T + (REV ? (size_t)(T - 1 - s) : (size_t)s)) * N + tid;
                if (a.yold) mb = max(mb, absdiff_bits(yn, __ldg(a.yold + vb)));
                a.y[vb] = yn;
            }
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
    asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
    __syncthreads();
    if (warp == 0) asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem), "r"(C::TMEM_COLS) : "memory");
    if (tid == 0) scan_epilogue(a.st);
}

}  // namespace deer
