// Cell + Jacobian + rhs (steps a1-a4) for n in {16, 32, 64} and the tiled input projection (a0).
//
// Both kernels are bound by the bytes they write (4 n^2 per position for J, 12 n per position
// for u), so the work is arranged for fully coalesced 128-bit stores and conflict-free shared
// memory reads; the small contractions [tile, n] x [n, 3n] run on the fp32 pipes with a 4-position
// register block per thread.
#pragma once
#include "common.cuh"

namespace deer {

template <int N> struct CellWide {
    static constexpr int THREADS = 256;
    static constexpr int P = 4;                         // positions per thread in the gate phase
    static constexpr int GROUPS = THREADS / N;          // position groups per tile
    static constexpr int PT = GROUPS * P;               // positions per tile
    static constexpr int HS = N + 4;                    // row stride of the h_prev tile (floats)
    static constexpr int CHUNKS = N * N / 4;            // float4 pieces of one Jacobian
    static constexpr int CPT = CHUNKS >= THREADS ? CHUNKS / THREADS : 1;   // pieces per thread
    static constexpr int PPAR = CHUNKS >= THREADS ? 1 : THREADS / CHUNKS;  // positions in parallel
    static constexpr size_t SMEM = sizeof(float) * (3 * N * N + 3 * N + PT * HS + 4 * PT * N);
};

// h_prev of the tile's positions -> shared memory rows of stride HS (zero rows past the end)
template <int N>
__device__ __forceinline__ void stage_h_prev(float *sH, const float *y, const float *y0, int T, size_t e0, int np, int tid)
{
    using C = CellWide<N>;
    for (int idx = tid; idx < C::PT * (N / 4); idx += C::THREADS) {
        const int p = idx / (N / 4), k4 = idx % (N / 4);
        float4 v = make_float4(0.f, 0.f, 0.f, 0.f);
        if (p < np) {
            const size_t e = e0 + p;
            size_t seq;
            const float *hp = seq_start(e, T, seq) ? y0 + seq * N : y + (e - 1) * N;
            v = *reinterpret_cast<const float4 *>(hp + 4 * k4);
        }
        *reinterpret_cast<float4 *>(sH + p * C::HS + 4 * k4) = v;
    }
}

// bias-free hidden projections of P positions for output row gi:  g*[q] = sum_k W_h*[gi][k] h_q[k]
template <int N>
__device__ __forceinline__ void gate_accumulate(float (&gr)[CellWide<N>::P], float (&gz)[CellWide<N>::P],
                                                float (&gq)[CellWide<N>::P], const float *sWT,
                                                const float *hrow, int gi)
{
    using C = CellWide<N>;
#pragma unroll
    for (int q = 0; q < C::P; ++q) { gr[q] = 0.0f; gz[q] = 0.0f; gq[q] = 0.0f; }
#pragma unroll 2
    for (int k = 0; k < N; k += 4) {
        float4 h4[C::P];
#pragma unroll
        for (int q = 0; q < C::P; ++q) h4[q] = *reinterpret_cast<const float4 *>(hrow + q * C::HS + k);
#pragma unroll
        for (int kk = 0; kk < 4; ++kk) {
            const float wr = sWT[(k + kk) * 3 * N + gi];
            const float wz = sWT[(k + kk) * 3 * N + N + gi];
            const float wn = sWT[(k + kk) * 3 * N + 2 * N + gi];
#pragma unroll
            for (int q = 0; q < C::P; ++q) {
                const float h = kk == 0 ? h4[q].x : kk == 1 ? h4[q].y : kk == 2 ? h4[q].z : h4[q].w;
                gr[q] = fmaf(wr, h, gr[q]);
                gz[q] = fmaf(wz, h, gz[q]);
                gq[q] = fmaf(wn, h, gq[q]);
            }
        }
    }
}

// Gate phase: thread (row i, group) accumulates the three hidden projections of its P positions
// from W_h^T in shared memory (lanes = consecutive rows: conflict-free) and h_prev broadcast
// from the staged tile; writes rhs = f - J h_prev using
//   J h = z.h + a_z.(W_hz h) + a_n r.(W_hn h) + a_n q r(1-r).(W_hr h)
// (the three products are the bias-free accumulators of the gate phase), and leaves the row
// coefficients {k_r, a_z, k_n, z} in shared memory.
// Jacobian phase: each thread owns fixed float4 pieces (row i, columns 4c..4c+3) of the three
// weight blocks in registers and streams  k_r W_hr + a_z W_hz + k_n W_hn + z I  for the tile's
// positions; a warp writes 512 contiguous bytes per store instruction.
template <int N>
__global__ void __launch_bounds__(256, (N <= 32) ? 4 : 0) cell_wide_kernel(CellArgs a)
{
    pdl_prologue();
    if (loop_ended(a.st)) return;
    using C = CellWide<N>;
    extern __shared__ __align__(16) float sm[];
    float *sWT = sm;                           // [N][3N]  W_h transposed: sWT[k*3N + g] = W_h[g][k]
    float *sB = sWT + 3 * N * N;               // [3N]
    float *sH = sB + 3 * N;                    // [PT][HS]
    float4 *sC = reinterpret_cast<float4 *>(sH + C::PT * C::HS);   // [PT][N] {k_r, a_z, k_n, z}

    const int tid = threadIdx.x;
    for (int idx = tid; idx < 3 * N * N; idx += C::THREADS) {
        const int g = idx / N, k = idx % N;
        sWT[k * 3 * N + g] = a.W_h[idx];
    }
    for (int idx = tid; idx < 3 * N; idx += C::THREADS) sB[idx] = a.b_h[idx];

    // Jacobian-phase weights: piece c of this thread is (row i, column block j4)
    float4 wR[C::CPT], wZ[C::CPT], wN[C::CPT];
    int dsel[C::CPT];
#pragma unroll
    for (int r = 0; r < C::CPT; ++r) {
        const int c = (tid + r * C::THREADS) % C::CHUNKS;
        const int i = c / (N / 4), j4 = c % (N / 4);
        wR[r] = *reinterpret_cast<const float4 *>(a.W_h + (size_t)i * N + 4 * j4);
        wZ[r] = *reinterpret_cast<const float4 *>(a.W_h + (size_t)(N + i) * N + 4 * j4);
        wN[r] = *reinterpret_cast<const float4 *>(a.W_h + (size_t)(2 * N + i) * N + 4 * j4);
        dsel[r] = (i >= 4 * j4 && i < 4 * j4 + 4) ? i - 4 * j4 : -1;
    }
    __syncthreads();

    const int gi = tid % N, grp = tid / N;
    const float bR = sB[gi], bZ = sB[N + gi], bN = sB[2 * N + gi];
    const size_t total = (size_t)a.B * a.T;
    const size_t ntiles = (total + C::PT - 1) / C::PT;

    for (size_t tile = blockIdx.x; tile < ntiles; tile += gridDim.x) {
        const size_t e0 = tile * C::PT;
        const int np = (int)((total - e0) < (size_t)C::PT ? (total - e0) : (size_t)C::PT);
        stage_h_prev<N>(sH, a.y, a.y0, a.T, e0, np, tid);
        __syncthreads();

        // ---- gate phase
        {
            float gr[C::P], gz[C::P], gq[C::P];
            const float *hrow = sH + (grp * C::P) * C::HS;
            float ur[C::P], uz[C::P], un[C::P];
#pragma unroll
            for (int q = 0; q < C::P; ++q) {
                const int p = grp * C::P + q;
                const float *ue = a.u + (e0 + (p < np ? p : 0)) * 3 * N;
                ur[q] = ue[gi]; uz[q] = ue[N + gi]; un[q] = ue[2 * N + gi];
            }
            gate_accumulate<N>(gr, gz, gq, sWT, hrow, gi);
#pragma unroll
            for (int q = 0; q < C::P; ++q) {
                const int p = grp * C::P + q;
                if (p < np) {
                    const size_t e = e0 + p;
                    const float qn = gq[q] + bN;                 // q = W_hn h + b_hn
                    const float r = sigmoidf_gate(ur[q] + (gr[q] + bR));
                    const float z = sigmoidf_gate(uz[q] + (gz[q] + bZ));
                    const float c = tanhf_gate(un[q] + r * qn);
                    const float hi = hrow[q * C::HS + gi];
                    const float f = (1.0f - z) * c + z * hi;
                    const float az = (hi - c) * z * (1.0f - z);
                    const float an = (1.0f - z) * (1.0f - c * c);
                    const float kr = an * qn * r * (1.0f - r);
                    const float kn = an * r;
                    if (a.coef_only) reinterpret_cast<float4 *>(a.J)[e * N + gi] = make_float4(kr, az, kn, z);
                    else sC[p * N + gi] = make_float4(kr, az, kn, z);
                    if (a.rhs) {
                        if (a.residual) {
                            a.rhs[e * N + gi] = f - a.y[e * N + gi];
                        } else {
                            float jh = z * hi;
                            jh = fmaf(az, gz[q], jh);
                            jh = fmaf(kn, gq[q], jh);
                            jh = fmaf(kr, gr[q], jh);
                            a.rhs[e * N + gi] = f - jh;
                        }
                    }
                }
            }
        }
        __syncthreads();

        // ---- Jacobian phase (not when only the coefficient rows are wanted)
        for (int p = tid / C::CHUNKS; p < (a.coef_only ? 0 : np); p += C::PPAR) {       // tid / CHUNKS == 0 when CPT >= 1 piece
            float *Je = a.J + (e0 + p) * (size_t)(N * N);
#pragma unroll
            for (int r = 0; r < C::CPT; ++r) {
                const int c = (tid + r * C::THREADS) % C::CHUNKS;
                const int i = c / (N / 4);
                const float4 k = sC[p * N + i];
                float4 v;
                v.x = fmaf(k.x, wR[r].x, fmaf(k.y, wZ[r].x, k.z * wN[r].x));
                v.y = fmaf(k.x, wR[r].y, fmaf(k.y, wZ[r].y, k.z * wN[r].y));
                v.z = fmaf(k.x, wR[r].z, fmaf(k.y, wZ[r].z, k.z * wN[r].z));
                v.w = fmaf(k.x, wR[r].w, fmaf(k.y, wZ[r].w, k.z * wN[r].w));
                if (dsel[r] == 0) v.x += k.w;
                if (dsel[r] == 1) v.y += k.w;
                if (dsel[r] == 2) v.z += k.w;
                if (dsel[r] == 3) v.w += k.w;
                reinterpret_cast<float4 *>(Je)[c] = v;
            }
        }
        __syncthreads();
    }
}

// ------------------------------------------------------------------ a0: u = x W_i^T + b_i, tiled
// (also dx = dG_i W_i of the VJP: the same product with the weights already in [input][output]
// order and no bias).  blockDim.x = n3 * G.  Thread (output g, group) keeps PP positions in registers; W_i^T sits in
// shared memory (lanes = consecutive outputs: conflict-free), x is staged per tile and read as a
// broadcast.  Loads of x and stores of u are coalesced.
constexpr int PROJ_PP = 8;

__global__ void __launch_bounds__(256) proj_tiled_kernel(const float *__restrict__ x, const float *__restrict__ W_i,
                                                         const float *__restrict__ b_i, float *__restrict__ u,
                                                         size_t N, int m, int n3, int G, int wt_given)
{
    extern __shared__ __align__(16) float smp[];
    float *sWT = smp;                    // [m][n3]
    float *sX = sWT + (size_t)m * n3;    // [G*PP][m+1]
    const int tid = threadIdx.x;
    const int nthr = n3 * G;
    const int PT = G * PROJ_PP;
    const int xs = m + 1;
    if (wt_given) {                      // weights already stored [m][n3]
        for (int idx = tid; idx < n3 * m; idx += blockDim.x) sWT[idx] = W_i[idx];
    } else {
        for (int idx = tid; idx < n3 * m; idx += blockDim.x) {
            const int g = idx / m, k = idx % m;
            sWT[k * n3 + g] = W_i[idx];
        }
    }
    const bool active = tid < nthr;
    const int g = active ? tid % n3 : 0, grp = active ? tid / n3 : 0;
    const float bias = b_i ? b_i[g] : 0.0f;
    const size_t ntiles = (N + PT - 1) / PT;
    for (size_t tile = blockIdx.x; tile < ntiles; tile += gridDim.x) {
        const size_t e0 = tile * PT;
        const int np = (int)((N - e0) < (size_t)PT ? (N - e0) : (size_t)PT);
        __syncthreads();
        for (int idx = tid; idx < PT * m; idx += blockDim.x) {
            const int p = idx / m, k = idx % m;
            sX[p * xs + k] = p < np ? x[e0 * m + idx] : 0.0f;
        }
        __syncthreads();
        if (!active) continue;
        float acc[PROJ_PP];
#pragma unroll
        for (int q = 0; q < PROJ_PP; ++q) acc[q] = bias;
        const float *xr = sX + (grp * PROJ_PP) * xs;
        for (int k = 0; k < m; ++k) {
            const float w = sWT[k * n3 + g];
#pragma unroll
            for (int q = 0; q < PROJ_PP; ++q) acc[q] = fmaf(w, xr[q * xs + k], acc[q]);
        }
#pragma unroll
        for (int q = 0; q < PROJ_PP; ++q) {
            const int p = grp * PROJ_PP + q;
            if (p < np) u[(e0 + p) * n3 + g] = acc[q];
        }
    }
}

}  // namespace deer
