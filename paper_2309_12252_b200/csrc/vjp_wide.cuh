// Cell VJP (step a8) for n in {16, 32, 64}: gate gradients with the gate phase of cell_wide.cuh,
// and the parameter-gradient contraction  dW = dG^T V  over all B*T positions on tensor cores.
#pragma once
#include "cell_wide.cuh"
#include "kernels_generic.cuh"
#include "scan_warp8.cuh"

namespace deer {

// dGi = [da_r, da_z, da_n], dGh = [da_r, da_z, dq] at every position (gates recomputed from u, y_prev).
template <int N>
__global__ void __launch_bounds__(256) vjp_cell_wide_kernel(VjpArgs a)
{
    using C = CellWide<N>;
    extern __shared__ __align__(16) float sm[];
    float *sWT = sm;                           // [N][3N]
    float *sB = sWT + 3 * N * N;               // [3N]
    float *sH = sB + 3 * N;                    // [PT][HS]
    const int tid = threadIdx.x;
    for (int idx = tid; idx < 3 * N * N; idx += C::THREADS) {
        const int g = idx / N, k = idx % N;
        sWT[k * 3 * N + g] = a.W_h[idx];
    }
    for (int idx = tid; idx < 3 * N; idx += C::THREADS) sB[idx] = a.b_h[idx];
    __syncthreads();
    const int gi = tid % N, grp = tid / N;
    const float bR = sB[gi], bZ = sB[N + gi], bN = sB[2 * N + gi];
    const size_t total = (size_t)a.B * a.T;
    const size_t ntiles = (total + C::PT - 1) / C::PT;
    for (size_t tile = blockIdx.x; tile < ntiles; tile += gridDim.x) {
        const size_t e0 = tile * C::PT;
        const int np = (int)((total - e0) < (size_t)C::PT ? (total - e0) : (size_t)C::PT);
        __syncthreads();
        stage_h_prev<N>(sH, a.y, a.y0, a.T, e0, np, tid);
        __syncthreads();
        float gr[C::P], gz[C::P], gq[C::P], ur[C::P], uz[C::P], un[C::P], lam[C::P];
        const float *hrow = sH + (grp * C::P) * C::HS;
#pragma unroll
        for (int q = 0; q < C::P; ++q) {
            const int p = grp * C::P + q;
            const size_t e = e0 + (p < np ? p : 0);
            const float *ue = a.u + e * 3 * N;
            ur[q] = ue[gi]; uz[q] = ue[N + gi]; un[q] = ue[2 * N + gi];
            lam[q] = a.lam[e * N + gi];
        }
        gate_accumulate<N>(gr, gz, gq, sWT, hrow, gi);
#pragma unroll
        for (int q = 0; q < C::P; ++q) {
            const int p = grp * C::P + q;
            if (p < np) {
                const size_t e = e0 + p;
                const float qn = gq[q] + bN;
                const float r = sigmoidf_gate(ur[q] + (gr[q] + bR));
                const float z = sigmoidf_gate(uz[q] + (gz[q] + bZ));
                const float c = tanhf_gate(un[q] + r * qn);
                const float hi = hrow[q * C::HS + gi];
                const float dan = lam[q] * (1.0f - z) * (1.0f - c * c);
                const float daz = lam[q] * (hi - c) * z * (1.0f - z);
                const float dar = dan * qn * r * (1.0f - r);
                const float dq = dan * r;
                float *gI = a.dGi + e * 3 * N, *gH = a.dGh + e * 3 * N;
                gI[gi] = dar; gI[N + gi] = daz; gI[2 * N + gi] = dan;
                gH[gi] = dar; gH[N + gi] = daz; gH[2 * N + gi] = dq;
            }
        }
    }
}

// Stage 1 of the deterministic parameter-gradient reduction on tensor cores.
//   out[g][k] = sum_e dG[e][g] V[e][k]   (k == K: bias column, V = 1)
// CTA (p, c) covers slice p of the positions and columns 64c .. 64c+63; warp w owns output rows
// 16w .. 16w+15 (rows past n3 are idle) and the chunk's column blocks.  The contraction index is the
// position: per step of 8 positions the A fragment is dG^T (rows = gates), the B fragments are V; both
// are read straight from global memory as 32-byte row segments.  Products use the 3 x TF32 split
// (fp32-level accuracy); the bias column is the running sum of the A fragment (chunk 0 writes it).
// blockDim.x = 32 * ceil(n3 / 16), gridDim.y = ceil(K / 64).
__global__ void __launch_bounds__(384) wgrad_mma_kernel(WgradArgs a)
{
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    const int g = lane >> 2, t = lane & 3;
    const int n3 = a.n3, K = a.K, K1 = K + 1;
    const int kb = 64 * blockIdx.y;
    const int nb = min(8, (K - kb + 7) >> 3);
    const size_t e0 = (size_t)blockIdx.x * a.slice;
    const size_t e1 = e0 + a.slice < a.N ? e0 + a.slice : a.N;
    float acc[8][4];
#pragma unroll
    for (int nn = 0; nn < 8; ++nn)
#pragma unroll
        for (int i = 0; i < 4; ++i) acc[nn][i] = 0.0f;
    float bs0 = 0.0f, bs1 = 0.0f;
    const int row = 16 * warp + g;
    const bool rv0 = row < n3, rv1 = row + 8 < n3;
    auto vrow = [&](size_t e) -> const float * {
        if (!a.shifted) return a.V + e * K;
        size_t seq;
        return seq_start(e, a.T, seq) ? a.y0 + seq * K : a.V + (e - 1) * K;
    };
#pragma unroll 1
    for (size_t e = e0; e < e1; e += 8) {
        const size_t p0 = e + t, p1 = e + t + 4;
        const bool v0 = p0 < e1, v1 = p1 < e1;
        float av[4];
        av[0] = (v0 && rv0) ? __ldg(a.dG + p0 * n3 + row) : 0.0f;
        av[1] = (v0 && rv1) ? __ldg(a.dG + p0 * n3 + row + 8) : 0.0f;
        av[2] = (v1 && rv0) ? __ldg(a.dG + p1 * n3 + row) : 0.0f;
        av[3] = (v1 && rv1) ? __ldg(a.dG + p1 * n3 + row + 8) : 0.0f;
        const float *r0 = v0 ? vrow(p0) : a.V, *r1 = v1 ? vrow(p1) : a.V;
        float bv[8][2];
#pragma unroll
        for (int nn = 0; nn < 8; ++nn) {
            const int col = kb + 8 * nn + g;
            const bool cv = nn < nb && col < K;
            bv[nn][0] = (cv && v0) ? __ldg(r0 + col) : 0.0f;
            bv[nn][1] = (cv && v1) ? __ldg(r1 + col) : 0.0f;
        }
        bs0 += av[0] + av[2];
        bs1 += av[1] + av[3];
        unsigned ah[4], al[4];
#pragma unroll
        for (int i = 0; i < 4; ++i) split_tf32(av[i], ah[i], al[i]);
#pragma unroll
        for (int nn = 0; nn < 8; ++nn) {
            if (nn < nb) {
                unsigned bh[2], bl[2];
                split_tf32(bv[nn][0], bh[0], bl[0]);
                split_tf32(bv[nn][1], bh[1], bl[1]);
                mma_tf32(acc[nn], al, bh, acc[nn]);
                mma_tf32(acc[nn], ah, bl, acc[nn]);
                mma_tf32(acc[nn], ah, bh, acc[nn]);
            }
        }
    }
    float *out = a.partial + (size_t)blockIdx.x * n3 * K1;
#pragma unroll
    for (int nn = 0; nn < 8; ++nn) {
        if (nn < nb) {
            const int col = kb + 8 * nn + 2 * t;
            if (col < K) {
                if (rv0) out[row * K1 + col] = acc[nn][0];
                if (rv1) out[(row + 8) * K1 + col] = acc[nn][2];
            }
            if (col + 1 < K) {
                if (rv0) out[row * K1 + col + 1] = acc[nn][1];
                if (rv1) out[(row + 8) * K1 + col + 1] = acc[nn][3];
            }
        }
    }
    if (blockIdx.y != 0) return;
    bs0 += __shfl_xor_sync(0xffffffffu, bs0, 1);
    bs0 += __shfl_xor_sync(0xffffffffu, bs0, 2);
    bs1 += __shfl_xor_sync(0xffffffffu, bs1, 1);
    bs1 += __shfl_xor_sync(0xffffffffu, bs1, 2);
    if (t == 0) {
        if (rv0) out[row * K1 + K] = bs0;
        if (rv1) out[(row + 8) * K1 + K] = bs1;
    }
}

// The same reduction with both operands staged through shared memory: the tiles of dG (WG_S positions x n3, one
// contiguous block) and of V (WG_S rows of the chunk's columns) arrive by 16-byte asynchronous copies in which
// consecutive lanes copy consecutive pieces -- full lines per instruction, where the direct 4-byte fragment loads above
// touch four rows with one sector each -- in a ring of WG_STAGES stages; the fragments are then read from shared memory
// (row strides = 8 mod 32 words: conflict-free).  Needs n3 % 4 == 0, K % 4 == 0 and 16-byte aligned operands.
constexpr int WG_S = 16, WG_STAGES = 3, WG_VS = 72;
__host__ __device__ inline int wgrad_gs(int n3) { return n3 + ((8 - n3 % 32) + 32) % 32; }
inline size_t wgrad_staged_smem(int n3) { return sizeof(float) * WG_STAGES * WG_S * (size_t)(wgrad_gs(n3) + WG_VS); }

__global__ void __launch_bounds__(384) wgrad_mma_staged_kernel(WgradArgs a)
{
    extern __shared__ __align__(16) float wg_sm[];
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5, nthr = blockDim.x;
    const int g = lane >> 2, t = lane & 3;
    const int n3 = a.n3, K = a.K, K1 = K + 1;
    const int GS = wgrad_gs(n3);
    const int kb = 64 * blockIdx.y;
    const int kc = min(64, K - kb);                    // columns of this chunk (a multiple of 4)
    const int nb = (kc + 7) >> 3;
    const size_t e0 = (size_t)blockIdx.x * a.slice;
    const size_t e1 = e0 + a.slice < a.N ? e0 + a.slice : a.N;
    const int nst = e1 > e0 ? (int)((e1 - e0 + WG_S - 1) / WG_S) : 0;
    float acc[8][4];
#pragma unroll
    for (int nn = 0; nn < 8; ++nn)
#pragma unroll
        for (int i = 0; i < 4; ++i) acc[nn][i] = 0.0f;
    float bs0 = 0.0f, bs1 = 0.0f;
    const int row = 16 * warp + g;
    const bool rv0 = row < n3, rv1 = row + 8 < n3;
    const int gq = n3 >> 2, vq = kc >> 2;              // 16-byte pieces per row of the two tiles
    auto issue = [&](int s) {
        if (s < nst) {
            float *sG = wg_sm + (size_t)(s % WG_STAGES) * WG_S * (GS + WG_VS), *sV = sG + WG_S * GS;
            const size_t pb = e0 + (size_t)s * WG_S;
            for (int c = tid; c < WG_S * gq; c += nthr) {
                const int r = c / gq, cc = c - r * gq;
                float *dst = sG + r * GS + 4 * cc;
                if (pb + r < e1) cp_async16(dst, a.dG + (pb + r) * n3 + 4 * cc);
                else *reinterpret_cast<float4 *>(dst) = make_float4(0.0f, 0.0f, 0.0f, 0.0f);
            }
            for (int c = tid; c < WG_S * vq; c += nthr) {
                const int r = c / vq, cc = c - r * vq;
                float *dst = sV + r * WG_VS + 4 * cc;
                const size_t e = pb + r;
                if (e < e1) {
                    const float *src = a.V + e * K;
                    if (a.shifted) {
                        size_t seq;
                        src = seq_start(e, a.T, seq) ? a.y0 + seq * K : a.V + (e - 1) * K;
                    }
                    cp_async16(dst, src + kb + 4 * cc);
                } else {
                    *reinterpret_cast<float4 *>(dst) = make_float4(0.0f, 0.0f, 0.0f, 0.0f);
                }
            }
        }
        cp_async_commit();
    };
#pragma unroll
    for (int s = 0; s < WG_STAGES - 1; ++s) issue(s);
#pragma unroll 1
    for (int s = 0; s < nst; ++s) {
        static_assert(WG_STAGES == 3, "the wait below leaves one group in flight");
        cp_async_wait_1();
        __syncthreads();                   // stage s landed for every thread; the stage of step s - 1 is free again
        issue(s + WG_STAGES - 1);
        const float *sG = wg_sm + (size_t)(s % WG_STAGES) * WG_S * (GS + WG_VS), *sV = sG + WG_S * GS;
#pragma unroll
        for (int sub = 0; sub < WG_S / 8; ++sub) {
            const float *g0 = sG + (8 * sub + t) * GS + row, *g1 = g0 + 4 * GS;
            float av[4];
            av[0] = rv0 ? g0[0] : 0.0f;
            av[1] = rv1 ? g0[8] : 0.0f;
            av[2] = rv0 ? g1[0] : 0.0f;
            av[3] = rv1 ? g1[8] : 0.0f;
            bs0 += av[0] + av[2];
            bs1 += av[1] + av[3];
            unsigned ah[4], al[4];
#pragma unroll
            for (int i = 0; i < 4; ++i) split_tf32(av[i], ah[i], al[i]);
            const float *v0 = sV + (8 * sub + t) * WG_VS + g, *v1 = v0 + 4 * WG_VS;
#pragma unroll
            for (int nn = 0; nn < 8; ++nn) {
                if (nn < nb) {
                    const bool cv = 8 * nn + g < kc;
                    unsigned bh[2], bl[2];
                    split_tf32(cv ? v0[8 * nn] : 0.0f, bh[0], bl[0]);
                    split_tf32(cv ? v1[8 * nn] : 0.0f, bh[1], bl[1]);
                    mma_tf32(acc[nn], al, bh, acc[nn]);
                    mma_tf32(acc[nn], ah, bl, acc[nn]);
                    mma_tf32(acc[nn], ah, bh, acc[nn]);
                }
            }
        }
    }
    cp_async_wait_0();
    float *out = a.partial + (size_t)blockIdx.x * n3 * K1;
#pragma unroll
    for (int nn = 0; nn < 8; ++nn) {
        if (nn < nb) {
            const int col = kb + 8 * nn + 2 * t;
            if (col < K) {
                if (rv0) out[row * K1 + col] = acc[nn][0];
                if (rv1) out[(row + 8) * K1 + col] = acc[nn][2];
            }
            if (col + 1 < K) {
                if (rv0) out[row * K1 + col + 1] = acc[nn][1];
                if (rv1) out[(row + 8) * K1 + col + 1] = acc[nn][3];
            }
        }
    }
    if (blockIdx.y != 0) return;
    bs0 += __shfl_xor_sync(0xffffffffu, bs0, 1);
    bs0 += __shfl_xor_sync(0xffffffffu, bs0, 2);
    bs1 += __shfl_xor_sync(0xffffffffu, bs1, 1);
    bs1 += __shfl_xor_sync(0xffffffffu, bs1, 2);
    if (t == 0) {
        if (rv0) out[row * K1 + K] = bs0;
        if (rv1) out[(row + 8) * K1 + K] = bs1;
    }
}

// ------------------------------------------------------------------ a0 / a8: dense affine map on tensor cores
//   out[e][c] = bias[c] + sum_k W(c,k) in[e][k],   W(c,k) = W[c*K + k]  (weights [out][in], the input
//   projection u = x W_i^T + b_i)  or  W[k*NOUT + c]  (WT_GIVEN: weights [in][out], dx = dG_i W_i).
// The batched [B*T, K] x [K, NOUT] contraction of the path: CTA = 8 warps, warp = 16 positions x all
// NOUT outputs, m16n8k8 TF32 MMAs issued three times on hi/lo splits (fp32-level accuracy).  The
// weights are split once per CTA into shared memory, rows padded so that the B-fragment reads are
// conflict-free; the contraction index is renamed so that a lane's two A values of a K step are
// adjacent in memory (one 8-byte load per row).  K % 8 == 0, NOUT % 8 == 0, NOUT <= 192.
template <int NB_MAX, bool WT_GIVEN>
__global__ void __launch_bounds__(256) affine_mma_kernel(const float *__restrict__ in, const float *__restrict__ W,
                                                         const float *__restrict__ bias, float *__restrict__ out,
                                                         size_t N, int K, int NOUT)
{
    extern __shared__ __align__(16) float smw[];
    const int NS = NOUT + 4;                  // row stride: 2 * NS = 8 (mod 32) words
    float *sBh = smw, *sBl = smw + (size_t)K * NS;
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const int g = lane >> 2, t = lane & 3;
    for (int idx = tid; idx < K * NOUT; idx += 256) {
        const int k = idx / NOUT, c = idx % NOUT;
        const float v = WT_GIVEN ? W[idx] : W[(size_t)c * K + k];
        sBh[k * NS + c] = v;
        sBl[k * NS + c] = v - __uint_as_float(__float_as_uint(v) & 0xffffe000u);
    }
    __syncthreads();
    const int nb = NOUT >> 3;
    const size_t ntiles = (N + 127) / 128;
    for (size_t tile = blockIdx.x; tile < ntiles; tile += gridDim.x) {
        const size_t p0 = tile * 128 + warp * 16;
        if (p0 >= N) continue;
        const size_t r0 = p0 + g, r1 = p0 + g + 8;
        const bool v0 = r0 < N, v1 = r1 < N;
        float acc[NB_MAX][4];
#pragma unroll
        for (int nn = 0; nn < NB_MAX; ++nn) {
            const float b0 = (bias && nn < nb) ? bias[8 * nn + 2 * t] : 0.0f, b1 = (bias && nn < nb) ? bias[8 * nn + 2 * t + 1] : 0.0f;
            acc[nn][0] = b0; acc[nn][1] = b1; acc[nn][2] = b0; acc[nn][3] = b1;
        }
        const float *a0p = in + (v0 ? r0 : 0) * K + 2 * t, *a1p = in + (v1 ? r1 : 0) * K + 2 * t;
        // the A values of the next K step are requested before the products of the current one
        float2 xn0 = v0 ? __ldg(reinterpret_cast<const float2 *>(a0p)) : make_float2(0.f, 0.f);
        float2 xn1 = v1 ? __ldg(reinterpret_cast<const float2 *>(a1p)) : make_float2(0.f, 0.f);
#pragma unroll 1
        for (int k0 = 0; k0 < K; k0 += 8) {
            // slots t and t+4 of the K step hold k0+2t and k0+2t+1
            const float2 x0 = xn0, x1 = xn1;
            if (k0 + 8 < K) {
                if (v0) xn0 = __ldg(reinterpret_cast<const float2 *>(a0p + k0 + 8));
                if (v1) xn1 = __ldg(reinterpret_cast<const float2 *>(a1p + k0 + 8));
            }
            unsigned ah[4], al[4];
            split_tf32(x0.x, ah[0], al[0]);      // a0: (row g,   slot t)
            split_tf32(x1.x, ah[1], al[1]);      // a1: (row g+8, slot t)
            split_tf32(x0.y, ah[2], al[2]);      // a2: (row g,   slot t+4)
            split_tf32(x1.y, ah[3], al[3]);      // a3: (row g+8, slot t+4)
            const float *bh0 = sBh + (k0 + 2 * t) * NS + g, *bl0 = sBl + (k0 + 2 * t) * NS + g;
#pragma unroll
            for (int nn = 0; nn < NB_MAX; ++nn) {
                if (nn < nb) {
                    unsigned bh[2], bl[2];
                    bh[0] = __float_as_uint(bh0[8 * nn]); bh[1] = __float_as_uint(bh0[8 * nn + NS]);
                    bl[0] = __float_as_uint(bl0[8 * nn]); bl[1] = __float_as_uint(bl0[8 * nn + NS]);
                    mma_tf32(acc[nn], al, bh, acc[nn]);
                    mma_tf32(acc[nn], ah, bl, acc[nn]);
                    mma_tf32(acc[nn], ah, bh, acc[nn]);
                }
            }
        }
#pragma unroll
        for (int nn = 0; nn < NB_MAX; ++nn) {
            if (nn < nb) {
                if (v0) *reinterpret_cast<float2 *>(out + r0 * NOUT + 8 * nn + 2 * t) = make_float2(acc[nn][0], acc[nn][1]);
                if (v1) *reinterpret_cast<float2 *>(out + r1 * NOUT + 8 * nn + 2 * t) = make_float2(acc[nn][2], acc[nn][3]);
            }
        }
    }
}

// ------------------------------------------------------------------ a1-a4 for n in {16, 32} when the scan builds J_t itself
// The cell as one tensor-core contraction with the gate math as its epilogue: [B*T, n] x [n, 3n]
// (h_prev times W_h^T; the input half u = x W_i^T + b_i comes from affine_mma_kernel, or, PROJ, is contracted here) as m16n8k8 TF32 MMAs
// issued three times on hi/lo splits, warp = 16 positions x all 3n outputs, weights split once per CTA
// into padded shared memory.  A lane's accumulator fragments hold, for its two positions and each of
// its columns i, the three bias-free products (W_hr h)_i, (W_hz h)_i, (W_hn h)_i -- the column blocks of
// the gates are n/8 apart -- so r, z, c, f, the coefficient row {k_r, a_z, k_n, z}_i and
// rhs_i = f_i - (J h)_i  (J h = z h + a_z W_hz h + k_n W_hn h + k_r W_hr h) follow in registers.
// Writes 16 n + 4 n bytes per position; no Jacobian.
template <int N, bool PROJ = false>
__global__ void __launch_bounds__(256, 2) cell_coef_mma_kernel(CellArgs a)
{
    pdl_prologue();
    if (loop_ended(a.st)) return;
    constexpr int NOUT = 3 * N, NB = NOUT / 8, NBG = N / 8;
    // B operands in shared memory as one 16-byte record per (pair of contraction rows, column):
    // {hi(W[2p][c]), hi(W[2p+1][c]), lo(W[2p][c]), lo(W[2p+1][c])} -- the four words a lane needs for one column block of
    // one K step, fetched by ONE 128-bit load; row stride NSQ = 2 (mod 8) records: the eight lanes of a quarter-warp
    // (two columns x four row pairs) read distinct bank groups
    constexpr int NSQ = NOUT + 2;
    extern __shared__ __align__(16) float smw[];
    float4 *sQ = reinterpret_cast<float4 *>(smw);
    float *sb = smw + 4 * (N / 2) * NSQ;
    // PROJ: the input projection is part of the same contraction ([B*T, m] x [m, 3n] with W_i^T, also 3 x TF32), so
    // neither a u buffer nor a projection pass exists: the r and z halves add into the hidden products' accumulators,
    // the candidate's input part keeps accumulators of its own (c = tanh(u_n + r q) needs the two apart).  Only with
    // the residual form (rhs = f - y), which does not need the bias-free hidden products.
    const int m = PROJ ? a.m : 0;
    float4 *sQi = reinterpret_cast<float4 *>(sb + 2 * NOUT);
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const int g = lane >> 2, t = lane & 3;
    auto tf32_lo = [](float v) { return v - __uint_as_float(__float_as_uint(v) & 0xffffe000u); };
    for (int idx = tid; idx < (N / 2) * NOUT; idx += 256) {
        const int kp = idx / NOUT, c = idx % NOUT;
        const float v0 = a.W_h[(size_t)c * N + 2 * kp], v1 = a.W_h[(size_t)c * N + 2 * kp + 1];
        sQ[kp * NSQ + c] = make_float4(v0, v1, tf32_lo(v0), tf32_lo(v1));
    }
    for (int idx = tid; idx < NOUT; idx += 256) { sb[idx] = a.b_h[idx]; sb[NOUT + idx] = PROJ ? a.b_i[idx] : 0.0f; }
    if constexpr (PROJ) {
        for (int idx = tid; idx < (m / 2) * NOUT; idx += 256) {
            const int kp = idx / NOUT, c = idx % NOUT;
            const float v0 = a.W_i[(size_t)c * m + 2 * kp], v1 = a.W_i[(size_t)c * m + 2 * kp + 1];
            sQi[kp * NSQ + c] = make_float4(v0, v1, tf32_lo(v0), tf32_lo(v1));
        }
    }
    __syncthreads();
    const size_t total = (size_t)a.B * a.T;
    const size_t ntiles = (total + 127) / 128;
    float4 *coef = reinterpret_cast<float4 *>(a.J);
    for (size_t tile = blockIdx.x; tile < ntiles; tile += gridDim.x) {
        const size_t p0 = tile * 128 + warp * 16;
        if (p0 >= total) continue;
        const size_t rr[2] = {p0 + g, p0 + g + 8};
        const bool vv[2] = {rr[0] < total, rr[1] < total};
        const float *hp[2];
#pragma unroll
        for (int h = 0; h < 2; ++h) {
            size_t seq = 0;
            hp[h] = a.y;
            if (vv[h]) hp[h] = seq_start(rr[h], a.T, seq) ? a.y0 + seq * N : a.y + (rr[h] - 1) * N;
        }
        float acc[NB][4];
#pragma unroll
        for (int nn = 0; nn < NB; ++nn) { acc[nn][0] = 0.0f; acc[nn][1] = 0.0f; acc[nn][2] = 0.0f; acc[nn][3] = 0.0f; }
        float accn[PROJ ? NBG : 1][4];                 // input part of the candidate gate (PROJ)
#pragma unroll
        for (int nn = 0; nn < (PROJ ? NBG : 1); ++nn) { accn[nn][0] = 0.0f; accn[nn][1] = 0.0f; accn[nn][2] = 0.0f; accn[nn][3] = 0.0f; }
#pragma unroll
        for (int k0 = 0; k0 < N; k0 += 8) {
            // slots t and t+4 of the K step hold k0+2t and k0+2t+1
            const float2 x0 = vv[0] ? __ldg(reinterpret_cast<const float2 *>(hp[0] + k0 + 2 * t)) : make_float2(0.f, 0.f);
            const float2 x1 = vv[1] ? __ldg(reinterpret_cast<const float2 *>(hp[1] + k0 + 2 * t)) : make_float2(0.f, 0.f);
            unsigned ah[4], al[4];
            split_tf32(x0.x, ah[0], al[0]);
            split_tf32(x1.x, ah[1], al[1]);
            split_tf32(x0.y, ah[2], al[2]);
            split_tf32(x1.y, ah[3], al[3]);
            const float4 *q0 = sQ + (k0 / 2 + t) * NSQ + g;
#pragma unroll
            for (int nn = 0; nn < NB; ++nn) {
                const float4 q = q0[8 * nn];
                const unsigned bh[2] = {__float_as_uint(q.x), __float_as_uint(q.y)}, bl[2] = {__float_as_uint(q.z), __float_as_uint(q.w)};
                mma_tf32(acc[nn], al, bh, acc[nn]);
                mma_tf32(acc[nn], ah, bl, acc[nn]);
                mma_tf32(acc[nn], ah, bh, acc[nn]);
            }
        }
        if constexpr (PROJ) {
            const float *xp0 = a.x + rr[0] * m, *xp1 = a.x + rr[1] * m;
#pragma unroll 2
            for (int k0 = 0; k0 < m; k0 += 8) {
                const float2 x0 = vv[0] ? __ldg(reinterpret_cast<const float2 *>(xp0 + k0 + 2 * t)) : make_float2(0.f, 0.f);
                const float2 x1 = vv[1] ? __ldg(reinterpret_cast<const float2 *>(xp1 + k0 + 2 * t)) : make_float2(0.f, 0.f);
                unsigned ah[4], al[4];
                split_tf32(x0.x, ah[0], al[0]);
                split_tf32(x1.x, ah[1], al[1]);
                split_tf32(x0.y, ah[2], al[2]);
                split_tf32(x1.y, ah[3], al[3]);
                const float4 *q0 = sQi + (k0 / 2 + t) * NSQ + g;
#pragma unroll
                for (int nn = 0; nn < NB; ++nn) {
                    const float4 q = q0[8 * nn];
                    const unsigned bh[2] = {__float_as_uint(q.x), __float_as_uint(q.y)}, bl[2] = {__float_as_uint(q.z), __float_as_uint(q.w)};
                    float (&dst)[4] = nn < 2 * NBG ? acc[nn] : accn[nn - 2 * NBG];
                    mma_tf32(dst, al, bh, dst);
                    mma_tf32(dst, ah, bl, dst);
                    mma_tf32(dst, ah, bh, dst);
                }
            }
        }
        // ---- epilogue: gates, coefficient rows, rhs for (position rr[h], columns 8nn+2t, 8nn+2t+1)
#pragma unroll
        for (int h = 0; h < 2; ++h) {
            if (!vv[h]) continue;
            const size_t e = rr[h];
            const float *ue = PROJ ? nullptr : a.u + e * NOUT;
#pragma unroll
            for (int nn = 0; nn < NBG; ++nn) {
                const int i0 = 8 * nn + 2 * t;
                float2 ur2 = make_float2(0.f, 0.f), uz2 = ur2, un2 = ur2;
                if constexpr (!PROJ) {
                    ur2 = __ldg(reinterpret_cast<const float2 *>(ue + i0));
                    uz2 = __ldg(reinterpret_cast<const float2 *>(ue + N + i0));
                    un2 = __ldg(reinterpret_cast<const float2 *>(ue + 2 * N + i0));
                } else {
                    ur2 = *reinterpret_cast<const float2 *>(sb + NOUT + i0);
                    uz2 = *reinterpret_cast<const float2 *>(sb + NOUT + N + i0);
                    un2 = fadd2(make_float2(accn[nn][2 * h], accn[nn][2 * h + 1]), *reinterpret_cast<const float2 *>(sb + NOUT + 2 * N + i0));
                }
                const float2 h2 = __ldg(reinterpret_cast<const float2 *>(hp[h] + i0));
                // the pair of columns i0, i0 + 1 as packed f32x2 arithmetic (half the instructions of two scalar passes)
                const float2 one = make_float2(1.0f, 1.0f), mone = make_float2(-1.0f, -1.0f);
                const float2 sr = make_float2(acc[nn][2 * h], acc[nn][2 * h + 1]);
                const float2 sz = make_float2(acc[nn + NBG][2 * h], acc[nn + NBG][2 * h + 1]);
                const float2 sq = make_float2(acc[nn + 2 * NBG][2 * h], acc[nn + 2 * NBG][2 * h + 1]);
                const float2 bR = *reinterpret_cast<const float2 *>(sb + i0), bZ = *reinterpret_cast<const float2 *>(sb + N + i0);
                const float2 qn = fadd2(sq, *reinterpret_cast<const float2 *>(sb + 2 * N + i0));   // q = W_hn h + b_hn
                const float2 r = sigmoid2_gate(fadd2(ur2, fadd2(sr, bR)));
                const float2 z = sigmoid2_gate(fadd2(uz2, fadd2(sz, bZ)));
                const float2 c = tanh2_gate(ffma2(r, qn, un2));
                const float2 omz = ffma2(z, mone, one), omr = ffma2(r, mone, one);
                const float2 f = ffma2(omz, c, fmul2(z, h2));
                const float2 az = fmul2(fmul2(ffma2(c, mone, h2), z), omz);
                const float2 an = fmul2(omz, ffma2(fmul2(c, mone), c, one));
                const float2 kr = fmul2(fmul2(fmul2(an, qn), r), omr);
                const float2 kn = fmul2(an, r);
                float4 cf2[2];
                cf2[0] = make_float4(kr.x, az.x, kn.x, z.x);
                cf2[1] = make_float4(kr.y, az.y, kn.y, z.y);
                float out_rhs[2];
                if (PROJ || a.residual) {
                    out_rhs[0] = f.x; out_rhs[1] = f.y;
                } else {
                    float2 jh = fmul2(z, h2);
                    jh = ffma2(az, sz, jh);
                    jh = ffma2(kn, sq, jh);
                    jh = ffma2(kr, sr, jh);
                    const float2 o = ffma2(jh, mone, f);
                    out_rhs[0] = o.x; out_rhs[1] = o.y;
                }
                // the rows of columns i0 and i0 + 1 are 32 contiguous bytes: one 256-bit store, so that the four lanes of a
                // position write one full line per instruction instead of eight half sectors
                st_global_v8(reinterpret_cast<float *>(coef + e * N + i0), cf2[0], cf2[1]);
                if (a.rhs && (PROJ || a.residual)) {
                    const float2 yc = __ldg(reinterpret_cast<const float2 *>(a.y + e * N + i0));
                    out_rhs[0] -= yc.x; out_rhs[1] -= yc.y;
                }
                if (a.rhs) *reinterpret_cast<float2 *>(a.rhs + e * N + i0) = make_float2(out_rhs[0], out_rhs[1]);
            }
        }
    }
}

}  // namespace deer
