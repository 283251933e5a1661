// Generic (any 1 <= n <= 64) kernels: input projection, cell + Jacobian + rhs,
// three-level chunked scan, cell VJP and the deterministic parameter-gradient
// reductions.  Simple shared-memory formulations; the tuned paths for
// n in {1,2,4,8} and the tensor-core paths replace the scan / cell kernels
// where they apply.
#pragma once
#include "common.cuh"

namespace deer {

constexpr int GEN_THREADS = 128;

// ------------------------------------------------------------------ a0: u = x W_i^T + b_i
__global__ void proj_kernel(const float *__restrict__ x, const float *__restrict__ W_i,
                            const float *__restrict__ b_i, float *__restrict__ u, size_t N, int m,
                            int n3)
{
    size_t idx = (size_t)blockIdx.x * blockDim.x + threadIdx.x;
    if (idx >= N * (size_t)n3) return;
    size_t e = idx / n3;
    int g = (int)(idx - e * n3);
    const float *xr = x + e * m;
    const float *wr = W_i + (size_t)g * m;
    float acc = b_i[g];
    for (int k = 0; k < m; ++k) acc = fmaf(wr[k], xr[k], acc);
    u[idx] = acc;
}

// ------------------------------------------------------------------ a1-a4: cell, Jacobian, rhs
// One thread per (position, output row).  Closed-form Jacobian
//   J = diag(z) + diag(a_z) W_hz + diag(a_n r) W_hn + diag(a_n q r (1-r)) W_hr.
__global__ void cell_kernel(CellArgs a)
{
    if (loop_ended(a.st)) return;
    extern __shared__ float sW[];          // W_h rows padded to n+1, then b_h
    const int n = a.n, ld = n + 1;
    float *sb = sW + 3 * n * ld;
    for (int i = threadIdx.x; i < 3 * n * n; i += blockDim.x) sW[(i / n) * ld + (i % n)] = a.W_h[i];
    for (int i = threadIdx.x; i < 3 * n; i += blockDim.x) sb[i] = a.b_h[i];
    __syncthreads();
    const int epb = blockDim.x / n;
    const int le = threadIdx.x / n, i = threadIdx.x % n;
    const size_t N = (size_t)a.B * a.T;
    const size_t e = (size_t)blockIdx.x * epb + le;
    if (le >= epb || e >= N) return;
    const int t = (int)(e % a.T);
    const size_t seq = e / a.T;
    const float *hp = (t == 0) ? a.y0 + seq * n : a.y + (e - 1) * n;
    float gr = sb[i], gz = sb[n + i], gq = sb[2 * n + i];
    for (int k = 0; k < n; ++k) {
        float h = hp[k];
        gr = fmaf(sW[i * ld + k], h, gr);
        gz = fmaf(sW[(n + i) * ld + k], h, gz);
        gq = fmaf(sW[(2 * n + i) * ld + k], h, gq);
    }
    const float *ue = a.u + e * 3 * n;
    float r = sigmoidf_acc(ue[i] + gr);
    float z = sigmoidf_acc(ue[n + i] + gz);
    float c = tanhf(ue[2 * n + i] + r * gq);
    float hi = hp[i];
    float f = (1.0f - z) * c + z * hi;
    float az = (hi - c) * z * (1.0f - z);
    float an = (1.0f - z) * (1.0f - c * c);
    float kr = an * gq * r * (1.0f - r);
    float kn = an * r;
    float acc = 0.0f;
    float *Jr = a.J + (e * n + i) * n;
    for (int j = 0; j < n; ++j) {
        float v = kr * sW[i * ld + j] + az * sW[(n + i) * ld + j] + kn * sW[(2 * n + i) * ld + j];
        if (j == i) v += z;
        Jr[j] = v;
        acc = fmaf(v, hp[j], acc);
    }
    if (a.rhs) a.rhs[e * n + i] = f - acc;
}

// Same computation for n in {1,2,4,8}: the thread's three weight rows live in registers, positions
// are visited with a grid stride, h_prev is read and the Jacobian row written with 128-bit accesses.
// M > 0: the input projection (a0) is done on the fly from x with the thread's 3 x M weights in
// registers (small input sizes: cheaper than a separate pass over u); M == 0: read u.
template <int N, int M>
__global__ void __launch_bounds__(256) cell_small_kernel(CellArgs a)
{
    pdl_prologue();
    if (loop_ended(a.st)) return;
    constexpr int EPB = 256 / N;                       // positions per block per step
    const int i = threadIdx.x % N, le = threadIdx.x / N;
    float wr[N], wz[N], wn[N];
#pragma unroll
    for (int k = 0; k < N; ++k) {
        wr[k] = a.W_h[i * N + k];
        wz[k] = a.W_h[(N + i) * N + k];
        wn[k] = a.W_h[(2 * N + i) * N + k];
    }
    const float br = a.b_h[i], bz = a.b_h[N + i], bn = a.b_h[2 * N + i];
    constexpr int MM = M > 0 ? M : 1;
    float vr[MM], vz[MM], vn[MM], cr = 0.0f, cz = 0.0f, cn = 0.0f;
    if constexpr (M > 0) {
#pragma unroll
        for (int k = 0; k < M; ++k) {
            vr[k] = a.W_i[i * M + k];
            vz[k] = a.W_i[(N + i) * M + k];
            vn[k] = a.W_i[(2 * N + i) * M + k];
        }
        cr = a.b_i[i]; cz = a.b_i[N + i]; cn = a.b_i[2 * N + i];
    }
    const size_t total = (size_t)a.B * a.T;
    // (seq, t) of the thread's position is carried along the grid-stride loop instead of divided out
    const size_t stride = (size_t)gridDim.x * EPB;
    const size_t stride_seq = stride / a.T;
    const unsigned stride_t = (unsigned)(stride - stride_seq * a.T);
    size_t e = (size_t)blockIdx.x * EPB + le;
    size_t seq = e / a.T;
    unsigned t = (unsigned)(e - seq * a.T);
    for (; e < total; e += stride, seq += stride_seq, t += stride_t) {
        if (t >= (unsigned)a.T) { t -= (unsigned)a.T; ++seq; }
        const bool first = t == 0u;
        const float *hp = first ? a.y0 + seq * N : a.y + (e - 1) * N;
        float h[N];
        if constexpr (N >= 4) {
#pragma unroll
            for (int v = 0; v < N / 4; ++v) {
                const float4 f = reinterpret_cast<const float4 *>(hp)[v];
                h[4 * v] = f.x; h[4 * v + 1] = f.y; h[4 * v + 2] = f.z; h[4 * v + 3] = f.w;
            }
        } else {
#pragma unroll
            for (int k = 0; k < N; ++k) h[k] = hp[k];
        }
        float sr = 0.0f, sz = 0.0f, sq = 0.0f;          // bias-free products W_h* h
#pragma unroll
        for (int k = 0; k < N; ++k) {
            sr = fmaf(wr[k], h[k], sr);
            sz = fmaf(wz[k], h[k], sz);
            sq = fmaf(wn[k], h[k], sq);
        }
        const float gr = sr + br, gz = sz + bz, gq = sq + bn;
        float ur, uz, un;
        if constexpr (M > 0) {
            const float *xe = a.x + e * M;
            ur = cr; uz = cz; un = cn;
#pragma unroll
            for (int k = 0; k < M; ++k) {
                const float xv = xe[k];
                ur = fmaf(vr[k], xv, ur); uz = fmaf(vz[k], xv, uz); un = fmaf(vn[k], xv, un);
            }
        } else {
            const float *ue = a.u + e * 3 * N;
            ur = ue[i]; uz = ue[N + i]; un = ue[2 * N + i];
        }
        const float r = sigmoidf_gate(ur + gr);
        const float z = sigmoidf_gate(uz + gz);
        const float c = tanhf_gate(un + r * gq);
        const float hi = hp[i];
        const float f = (1.0f - z) * c + z * hi;
        const float az = (hi - c) * z * (1.0f - z);
        const float an = (1.0f - z) * (1.0f - c * c);
        const float kr = an * gq * r * (1.0f - r);
        const float kn = an * r;
        float v[N];
#pragma unroll
        for (int j = 0; j < N; ++j) {
            v[j] = kr * wr[j] + az * wz[j] + kn * wn[j];
            if (j == i) v[j] += z;
        }
        // J h = z h_i + a_z (W_hz h)_i + k_n (W_hn h)_i + k_r (W_hr h)_i, from the gate accumulators
        const float acc = fmaf(kr, sr, fmaf(kn, sq, fmaf(az, sz, z * hi)));
        float *Jr = a.J + (e * N + i) * N;
        if constexpr (N >= 4) {
#pragma unroll
            for (int q = 0; q < N / 4; ++q)
                reinterpret_cast<float4 *>(Jr)[q] = make_float4(v[4 * q], v[4 * q + 1], v[4 * q + 2], v[4 * q + 3]);
        } else if constexpr (N == 2) {
            *reinterpret_cast<float2 *>(Jr) = make_float2(v[0], v[1]);
        } else {
            Jr[0] = v[0];
        }
        if (a.rhs) a.rhs[e * N + i] = f - acc;
    }
}

// ------------------------------------------------------------------ a5: generic chunked scan
__device__ __forceinline__ void gen_load_M(float *dst, const ScanArgs &a, size_t seq, int s)
{
    const int n = a.n, nn = n * n;
    if (!a.reverse) {
        const float *src = a.J + (seq * a.T + s) * nn;
        for (int i = threadIdx.x; i < nn; i += blockDim.x) dst[i] = src[i];
    } else if (s == 0) {
        for (int i = threadIdx.x; i < nn; i += blockDim.x) dst[i] = (i / n == i % n) ? 1.0f : 0.0f;
    } else {
        const float *src = a.J + (seq * a.T + (a.T - s)) * nn;     // J[t+1], t = T-1-s
        for (int i = threadIdx.x; i < nn; i += blockDim.x) dst[(i % n) * n + (i / n)] = src[i];
    }
}

__device__ __forceinline__ size_t gen_vec_index(const ScanArgs &a, size_t seq, int s, int i)
{
    int t = a.reverse ? a.T - 1 - s : s;
    return (seq * a.T + t) * a.n + i;
}

// level 1: one CTA folds one chunk into (A, beta), later positions multiplying on the left.
__global__ void gen_reduce_kernel(ScanArgs a)
{
    if (loop_ended(a.st)) return;
    extern __shared__ float sm[];
    const int n = a.n, nn = n * n;
    float *Jt = sm, *A = sm + nn, *A2 = sm + 2 * nn, *be = sm + 3 * nn, *be2 = be + n;
    const int c = blockIdx.x;
    const size_t seq = blockIdx.y;
    const int s0 = c * a.L, s1 = min(a.T, s0 + a.L);
    gen_load_M(A, a, seq, s0);
    if (threadIdx.x < n) be[threadIdx.x] = a.b[gen_vec_index(a, seq, s0, threadIdx.x)];
    __syncthreads();
    for (int s = s0 + 1; s < s1; ++s) {
        gen_load_M(Jt, a, seq, s);
        __syncthreads();
        for (int idx = threadIdx.x; idx < nn; idx += blockDim.x) {
            int i = idx / n, j = idx % n;
            float acc = 0.0f;
            for (int k = 0; k < n; ++k) acc = fmaf(Jt[i * n + k], A[k * n + j], acc);
            A2[idx] = acc;
        }
        if (threadIdx.x < n) {
            float acc = a.b[gen_vec_index(a, seq, s, threadIdx.x)];
            for (int k = 0; k < n; ++k) acc = fmaf(Jt[threadIdx.x * n + k], be[k], acc);
            be2[threadIdx.x] = acc;
        }
        __syncthreads();
        float *tmp = A; A = A2; A2 = tmp;
        tmp = be; be = be2; be2 = tmp;
    }
    float *oA = a.carA + (seq * a.nch + c) * nn;
    for (int i = threadIdx.x; i < nn; i += blockDim.x) oA[i] = A[i];
    if (threadIdx.x < n) a.carB[(seq * a.nch + c) * n + threadIdx.x] = be[threadIdx.x];
}

// level 2: one CTA per sequence walks the chunk aggregates in order.
__global__ void gen_carry_kernel(ScanArgs a)
{
    if (loop_ended(a.st)) return;
    extern __shared__ float sm[];
    const int n = a.n, nn = n * n;
    float *Am = sm, *Y = sm + nn;
    const size_t seq = blockIdx.x;
    if (threadIdx.x < n) Y[threadIdx.x] = a.y0 ? a.y0[seq * n + threadIdx.x] : 0.0f;
    __syncthreads();
    for (int c = 0; c < a.nch; ++c) {
        if (threadIdx.x < n) a.starts[(seq * a.nch + c) * n + threadIdx.x] = Y[threadIdx.x];
        if (c == a.nch - 1) break;
        const float *src = a.carA + (seq * a.nch + c) * nn;
        for (int i = threadIdx.x; i < nn; i += blockDim.x) Am[i] = src[i];
        __syncthreads();
        float v = 0.0f;
        if (threadIdx.x < n) {
            v = a.carB[(seq * a.nch + c) * n + threadIdx.x];
            for (int k = 0; k < n; ++k) v = fmaf(Am[threadIdx.x * n + k], Y[k], v);
        }
        __syncthreads();
        if (threadIdx.x < n) Y[threadIdx.x] = v;
        __syncthreads();
    }
}

// level 3: one CTA replays its chunk from the entering state, writes y and the max deviation.
__global__ void gen_apply_kernel(ScanArgs a)
{
    if (loop_ended(a.st)) return;
    extern __shared__ float sm[];
    const int n = a.n, nn = n * n;
    float *Jt = sm, *Y = sm + nn;
    const int c = blockIdx.x;
    const size_t seq = blockIdx.y;
    const int s0 = c * a.L, s1 = min(a.T, s0 + a.L);
    if (threadIdx.x < n) Y[threadIdx.x] = a.starts[(seq * a.nch + c) * n + threadIdx.x];
    unsigned mb = 0;
    for (int s = s0; s < s1; ++s) {
        gen_load_M(Jt, a, seq, s);
        __syncthreads();
        float v = 0.0f;
        size_t idx = 0;
        if (threadIdx.x < n) {
            idx = gen_vec_index(a, seq, s, threadIdx.x);
            v = a.b[idx];
            for (int k = 0; k < n; ++k) v = fmaf(Jt[threadIdx.x * n + k], Y[k], v);
        }
        __syncthreads();
        if (threadIdx.x < n) {
            Y[threadIdx.x] = v;
            if (a.yold) mb = max(mb, absdiff_bits(v, a.yold[idx]));
            a.y[idx] = v;
        }
    }
    if (a.yold) {
        for (int o = 16; o > 0; o >>= 1) mb = max(mb, __shfl_xor_sync(0xffffffffu, mb, o));
        if ((threadIdx.x & 31) == 0 && mb) atomicMax(&a.st->err_bits, mb);
    }
}

// ------------------------------------------------------------------ a6: loop control on the device
// Clears the single-pass scan's words (tile flags, entering states, counters) before the first scan
// on a workspace; the scans leave them cleared.
__global__ void scan_prep_kernel(StatusBlock *st, unsigned *flags, size_t nflags,
                                 unsigned long long *starts, size_t nstarts,
                                 unsigned long long *agg_words, size_t nagg_words)
{
    if (loop_ended(st)) return;
    const size_t stride = (size_t)gridDim.x * blockDim.x;
    const size_t i0 = (size_t)blockIdx.x * blockDim.x + threadIdx.x;
    for (size_t i = i0; i < nflags; i += stride) flags[i] = 0u;
    for (size_t i = i0; i < nstarts; i += stride) starts[i] = 0ull;
    for (size_t i = i0; i < nagg_words; i += stride) agg_words[i] = 0ull;
    if (i0 == 0) { st->tile_counter = 0u; st->role_counter = 0u; st->exit_counter = 0u; }
}

// Everything an evaluation needs before its first body, in one launch: the status block (loop
// control state, passed by value), the zero initial guess, and the cleared exchange words and
// counters of the single-pass scan.
struct EvalBeginArgs {
    float *y; size_t ny;                         // initial guess to zero (nullptr: warm start)
    unsigned *flags; size_t nflags;              // single-pass scan words (nullptr / 0 when not used)
    unsigned long long *starts; size_t nstarts;
    unsigned long long *agg_words; size_t nagg_words;
};
__global__ void eval_begin_kernel(StatusBlock *st, StatusBlock init, EvalBeginArgs e)
{
    const size_t stride = (size_t)gridDim.x * blockDim.x;
    const size_t i0 = (size_t)blockIdx.x * blockDim.x + threadIdx.x;
    if (i0 == 0) *st = init;
    if (e.y) {
        if (((uintptr_t)e.y & 15) == 0) {
            float4 *y4 = reinterpret_cast<float4 *>(e.y);
            const size_t n4 = e.ny / 4;
            for (size_t i = i0; i < n4; i += stride) y4[i] = make_float4(0.0f, 0.0f, 0.0f, 0.0f);
            for (size_t i = 4 * n4 + i0; i < e.ny; i += stride) e.y[i] = 0.0f;
        } else {
            for (size_t i = i0; i < e.ny; i += stride) e.y[i] = 0.0f;
        }
    }
    for (size_t i = i0; i < e.nflags; i += stride) e.flags[i] = 0u;
    for (size_t i = i0; i < e.nstarts; i += stride) e.starts[i] = 0ull;
    for (size_t i = i0; i < e.nagg_words; i += stride) e.agg_words[i] = 0ull;
}

// After an odd number of bodies the current iterate sits in the workspace copy: bring it into the
// caller's buffer on the device, without the host having to know the count (the buffer it overwrites
// is the one the next body, if any, overwrites anyway).  Runs whether or not the loop has ended.
__global__ void result_select_kernel(const StatusBlock *st, float *y, const float *yalt, size_t ny)
{
    if ((st->iters & 1) == 0) return;
    const size_t stride = (size_t)gridDim.x * blockDim.x;
    const size_t i0 = (size_t)blockIdx.x * blockDim.x + threadIdx.x;
    if ((((uintptr_t)y | (uintptr_t)yalt) & 15) == 0) {
        const size_t n4 = ny / 4;
        for (size_t i = i0; i < n4; i += stride) reinterpret_cast<float4 *>(y)[i] = reinterpret_cast<const float4 *>(yalt)[i];
        for (size_t i = 4 * n4 + i0; i < ny; i += stride) y[i] = yalt[i];
    } else {
        for (size_t i = i0; i < ny; i += stride) y[i] = yalt[i];
    }
}

// Diagnostics of the last body (one CTA per sequence): key[b] = max |y_new - y_old| over the sequence
// as float bits in the upper word, and 0xffffffff - (index within the sequence of its first occurrence)
// in the lower word, so that an integer max gives the largest deviation and, among equals, the
// smallest index.  Pure function of the two iterates: identical across runs.
__global__ void __launch_bounds__(256) err_diag_kernel(const float *__restrict__ ynew, const float *__restrict__ yold,
                                                        size_t per_seq, unsigned long long *__restrict__ key)
{
    __shared__ unsigned long long red[8];
    const size_t base = (size_t)blockIdx.x * per_seq;
    unsigned long long best = 0ull;
    for (size_t i = threadIdx.x; i < per_seq; i += blockDim.x) {
        const unsigned long long k = ((unsigned long long)absdiff_bits(ynew[base + i], yold[base + i]) << 32) |
                                     (unsigned long long)(0xffffffffu - (unsigned)i);
        best = k > best ? k : best;
    }
#pragma unroll
    for (int d = 16; d > 0; d >>= 1) {
        const unsigned long long o = __shfl_xor_sync(0xffffffffu, best, d);
        best = o > best ? o : best;
    }
    if ((threadIdx.x & 31) == 0) red[threadIdx.x >> 5] = best;
    __syncthreads();
    if (threadIdx.x == 0) {
        for (int w = 1; w < 8; ++w) best = red[w] > best ? red[w] : best;
        key[blockIdx.x] = best;
    }
}

// Loop control as a launch of its own (used when a body's scan ran on the generic kernels).
__global__ void newton_control_kernel(StatusBlock *st, float tol, int max_iter, float *trace)
{
    if (loop_ended(st)) return;
    newton_decide(st, tol, max_iter, trace);
}

// ------------------------------------------------------------------ a8: cell VJP
struct VjpArgs {
    const float *W_h, *b_h, *u, *y, *y0, *lam;   // lam [B,T,n] = dL/df at every position
    float *dGi, *dGh;                            // [B,T,3n] gradients w.r.t. u and w.r.t. W_h h + b_h
    int B, T, n;
};

__global__ void vjp_cell_kernel(VjpArgs a)
{
    extern __shared__ float sW[];
    const int n = a.n, ld = n + 1;
    float *sb = sW + 3 * n * ld;
    for (int i = threadIdx.x; i < 3 * n * n; i += blockDim.x) sW[(i / n) * ld + (i % n)] = a.W_h[i];
    for (int i = threadIdx.x; i < 3 * n; i += blockDim.x) sb[i] = a.b_h[i];
    __syncthreads();
    const int epb = blockDim.x / n;
    const int le = threadIdx.x / n, i = threadIdx.x % n;
    const size_t N = (size_t)a.B * a.T;
    const size_t e = (size_t)blockIdx.x * epb + le;
    if (le >= epb || e >= N) return;
    const int t = (int)(e % a.T);
    const size_t seq = e / a.T;
    const float *hp = (t == 0) ? a.y0 + seq * n : a.y + (e - 1) * n;
    float gr = sb[i], gz = sb[n + i], gq = sb[2 * n + i];
    for (int k = 0; k < n; ++k) {
        float h = hp[k];
        gr = fmaf(sW[i * ld + k], h, gr);
        gz = fmaf(sW[(n + i) * ld + k], h, gz);
        gq = fmaf(sW[(2 * n + i) * ld + k], h, gq);
    }
    const float *ue = a.u + e * 3 * n;
    float r = sigmoidf_acc(ue[i] + gr);
    float z = sigmoidf_acc(ue[n + i] + gz);
    float c = tanhf(ue[2 * n + i] + r * gq);
    float l = a.lam[e * n + i];
    float dan = l * (1.0f - z) * (1.0f - c * c);
    float daz = l * (hp[i] - c) * z * (1.0f - z);
    float dar = dan * gq * r * (1.0f - r);
    float dq = dan * r;
    float *gi = a.dGi + e * 3 * n, *gh = a.dGh + e * 3 * n;
    gi[i] = dar; gi[n + i] = daz; gi[2 * n + i] = dan;
    gh[i] = dar; gh[n + i] = daz; gh[2 * n + i] = dq;
}

// ------------------------------------------------------------------ a8 for small n: cell VJP and reductions in one pass
// n in {1,2,4,8}, m in {1,2,4,8} (Eq. 7 applied to the GRU; App. B.1).  One thread per (position, row i), as
// in cell_small_kernel: gates from h_prev and x (projection on the fly), then with lam = dL/df at the position
//   d_an = lam (1-z)(1-c^2),  d_az = lam (h_i - c) z (1-z),  d_ar = d_an q r (1-r),  d_q = d_an r
// (the gradients w.r.t. the three input-side and hidden-side pre-activations of row i), accumulated
// in registers straight into this thread's share of dW_i, dW_h, db_i, db_h -- no per-position gradient
// arrays exist -- and dx = W_i^T dG_i reduced over the rows of the position by shuffles.
// CTA p then adds its threads' sums in thread order and writes slice p of the two-stage reduction
// (stage 2: wgrad_final_kernel), so the result is bit-reproducible.
struct VjpSmallArgs {
    const float *W_h, *b_h, *W_i, *b_i, *x, *y, *y0, *lam;
    float *dx;                 // [B,T,m] or nullptr
    float *partial_i;          // [P][3n*(m+1)]
    float *partial_h;          // [P][3n*(n+1)]
    int B, T;
};

template <int N, int M>
__global__ void __launch_bounds__(256, 2) vjp_small_kernel(VjpSmallArgs a)
{
    constexpr int EPB = 256 / N;                       // positions per block per step
    constexpr int VI = 3 * (M + 1), VH = 3 * (N + 1), VALS = VI + VH;
    extern __shared__ float red[];                     // [256][VALS + 1]
    const int i = threadIdx.x % N, le = threadIdx.x / N;
    float wr[N], wz[N], wn[N], vr[M], vz[M], vn[M];
#pragma unroll
    for (int k = 0; k < N; ++k) {
        wr[k] = a.W_h[i * N + k];
        wz[k] = a.W_h[(N + i) * N + k];
        wn[k] = a.W_h[(2 * N + i) * N + k];
    }
#pragma unroll
    for (int k = 0; k < M; ++k) {
        vr[k] = a.W_i[i * M + k];
        vz[k] = a.W_i[(N + i) * M + k];
        vn[k] = a.W_i[(2 * N + i) * M + k];
    }
    const float br = a.b_h[i], bz = a.b_h[N + i], bn = a.b_h[2 * N + i];
    const float cr = a.b_i[i], cz = a.b_i[N + i], cn = a.b_i[2 * N + i];
    float ai[3][M + 1], ah[3][N + 1];
#pragma unroll
    for (int g = 0; g < 3; ++g) {
#pragma unroll
        for (int k = 0; k <= M; ++k) ai[g][k] = 0.0f;
#pragma unroll
        for (int k = 0; k <= N; ++k) ah[g][k] = 0.0f;
    }
    const size_t total = (size_t)a.B * a.T;
    const size_t stride = (size_t)gridDim.x * EPB;
    const size_t stride_seq = stride / a.T;
    const unsigned stride_t = (unsigned)(stride - stride_seq * a.T);
    size_t e = (size_t)blockIdx.x * EPB + le;
    size_t seq = e / a.T;
    unsigned t = (unsigned)(e - seq * a.T);
    // (every thread of a warp runs the same number of iterations when it shuffles: the loop bound is
    // taken on the position of the warp's first row group, and late positions are masked)
    for (; ; e += stride, seq += stride_seq, t += stride_t) {
        if (t >= (unsigned)a.T) { t -= (unsigned)a.T; ++seq; }
        const bool in = e < total;
        if (!__any_sync(0xffffffffu, in)) break;
        float h[N], xv[M], l = 0.0f, hi = 0.0f;
#pragma unroll
        for (int k = 0; k < N; ++k) h[k] = 0.0f;
#pragma unroll
        for (int k = 0; k < M; ++k) xv[k] = 0.0f;
        if (in) {
            const float *hp = (t == 0u) ? a.y0 + seq * N : a.y + (e - 1) * N;
#pragma unroll
            for (int k = 0; k < N; ++k) h[k] = hp[k];
#pragma unroll
            for (int k = 0; k < M; ++k) xv[k] = a.x[e * M + k];
            l = a.lam[e * N + i];
            hi = hp[i];
        }
        float gr = br, gz = bz, gq = bn, ur = cr, uz = cz, un = cn;
#pragma unroll
        for (int k = 0; k < N; ++k) {
            gr = fmaf(wr[k], h[k], gr);
            gz = fmaf(wz[k], h[k], gz);
            gq = fmaf(wn[k], h[k], gq);
        }
#pragma unroll
        for (int k = 0; k < M; ++k) {
            ur = fmaf(vr[k], xv[k], ur); uz = fmaf(vz[k], xv[k], uz); un = fmaf(vn[k], xv[k], un);
        }
        const float r = sigmoidf_gate(ur + gr);          // the activations of the forward small-n cell
        const float z = sigmoidf_gate(uz + gz);
        const float c = tanhf_gate(un + r * gq);
        const float dan = l * (1.0f - z) * (1.0f - c * c);
        const float daz = l * (hi - c) * z * (1.0f - z);
        const float dar = dan * gq * r * (1.0f - r);
        const float dq = dan * r;
#pragma unroll
        for (int k = 0; k < M; ++k) {
            ai[0][k] = fmaf(dar, xv[k], ai[0][k]); ai[1][k] = fmaf(daz, xv[k], ai[1][k]); ai[2][k] = fmaf(dan, xv[k], ai[2][k]);
        }
        ai[0][M] += dar; ai[1][M] += daz; ai[2][M] += dan;
#pragma unroll
        for (int k = 0; k < N; ++k) {
            ah[0][k] = fmaf(dar, h[k], ah[0][k]); ah[1][k] = fmaf(daz, h[k], ah[1][k]); ah[2][k] = fmaf(dq, h[k], ah[2][k]);
        }
        ah[0][N] += dar; ah[1][N] += daz; ah[2][N] += dq;
        if (a.dx) {
            float pk[M];
#pragma unroll
            for (int k = 0; k < M; ++k) {
                pk[k] = fmaf(vr[k], dar, fmaf(vz[k], daz, vn[k] * dan));
#pragma unroll
                for (int d = 1; d < N; d <<= 1) pk[k] += __shfl_xor_sync(0xffffffffu, pk[k], d);
            }
            if (in && i == 0) {
#pragma unroll
                for (int k = 0; k < M; ++k) a.dx[e * M + k] = pk[k];
            }
        }
    }
    // CTA reduction in thread order: thread (le, i) -> red[tid][...]; output (row i, value v) adds le = 0 .. EPB-1
    float *mine = red + threadIdx.x * (VALS + 1);
#pragma unroll
    for (int g = 0; g < 3; ++g) {
#pragma unroll
        for (int k = 0; k <= M; ++k) mine[g * (M + 1) + k] = ai[g][k];
#pragma unroll
        for (int k = 0; k <= N; ++k) mine[VI + g * (N + 1) + k] = ah[g][k];
    }
    __syncthreads();
    for (int o = threadIdx.x; o < N * VALS; o += blockDim.x) {
        const int row = o / VALS, v = o - row * VALS;
        float s = 0.0f;
        for (int q = 0; q < EPB; ++q) s += red[(q * N + row) * (VALS + 1) + v];
        if (v < VI) {
            const int g = v / (M + 1), k = v - g * (M + 1);
            a.partial_i[(size_t)blockIdx.x * (3 * N * (M + 1)) + (g * N + row) * (M + 1) + k] = s;
        } else {
            const int vv = v - VI, g = vv / (N + 1), k = vv - g * (N + 1);
            a.partial_h[(size_t)blockIdx.x * (3 * N * (N + 1)) + (g * N + row) * (N + 1) + k] = s;
        }
    }
}

// dx[e][k] = sum_g W_i[g][k] dGi[e][g]
__global__ void vjp_dx_kernel(const float *__restrict__ dGi, const float *__restrict__ W_i,
                              float *__restrict__ dx, size_t N, int m, int n3)
{
    size_t idx = (size_t)blockIdx.x * blockDim.x + threadIdx.x;
    if (idx >= N * (size_t)m) return;
    size_t e = idx / m;
    int k = (int)(idx - e * m);
    const float *g = dGi + e * n3;
    float acc = 0.0f;
    for (int j = 0; j < n3; ++j) acc = fmaf(W_i[(size_t)j * m + k], g[j], acc);
    dx[idx] = acc;
}

// dy0[b][j] = sum_i J[b][0][i][j] lam[b][0][i]
__global__ void vjp_dy0_kernel(const float *__restrict__ J, const float *__restrict__ lam,
                               float *__restrict__ dy0, int B, int T, int n)
{
    int idx = blockIdx.x * blockDim.x + threadIdx.x;
    if (idx >= B * n) return;
    int seq = idx / n, j = idx % n;
    const float *J0 = J + (size_t)seq * T * n * n;
    const float *l0 = lam + (size_t)seq * T * n;
    float acc = 0.0f;
    for (int i = 0; i < n; ++i) acc = fmaf(J0[i * n + j], l0[i], acc);
    dy0[idx] = acc;
}

// the same from the coefficient rows {k_r, a_z, k_n, z}[n] of position 0 (J = diag(k_r) W_hr + diag(a_z) W_hz +
// diag(k_n) W_hn + diag(z), evaluated in the order of the cell's Jacobian phase)
__global__ void vjp_dy0_coef_kernel(const float *__restrict__ coef, const float *__restrict__ W_h,
                                    const float *__restrict__ lam, float *__restrict__ dy0, int B, int T, int n)
{
    int idx = blockIdx.x * blockDim.x + threadIdx.x;
    if (idx >= B * n) return;
    int seq = idx / n, j = idx % n;
    const float4 *c0 = reinterpret_cast<const float4 *>(coef) + (size_t)seq * T * n;
    const float *l0 = lam + (size_t)seq * T * n;
    float acc = 0.0f;
    for (int i = 0; i < n; ++i) {
        const float4 k = c0[i];
        float v = fmaf(k.x, W_h[(size_t)i * n + j], fmaf(k.y, W_h[(size_t)(n + i) * n + j], k.z * W_h[(size_t)(2 * n + i) * n + j]));
        if (i == j) v += k.w;
        acc = fmaf(v, l0[i], acc);
    }
    dy0[idx] = acc;
}

// Deterministic two-stage reduction  out[g][k] = sum_e dG[e][g] * V[e][k]  (k == K: bias, V = 1).
// Stage 1: CTA (p, oy) accumulates 256 outputs over slice p of the positions, in position order.
struct WgradArgs {
    const float *dG;     // [N, n3]
    const float *V;      // [N, K]; if shifted: row e is y[e-1] (y0 at t = 0)
    const float *y0;
    int shifted, T, n3, K, tile;
    size_t N, slice;
    float *partial;      // [P][n3*(K+1)]
};

__global__ void wgrad_partial_kernel(WgradArgs a)
{
    extern __shared__ float sm[];
    const int K1 = a.K + 1, outs = a.n3 * K1;
    float *gt = sm, *vt = sm + a.tile * a.n3;
    const int o = blockIdx.y * blockDim.x + threadIdx.x;
    const bool valid = o < outs;
    const int g = valid ? o / K1 : 0, k = valid ? o % K1 : 0;
    const size_t e0 = (size_t)blockIdx.x * a.slice;
    const size_t e1 = min(a.N, e0 + a.slice);
    float acc = 0.0f;
    for (size_t base = e0; base < e1; base += a.tile) {
        const int cnt = (int)min((size_t)a.tile, e1 - base);
        for (int i = threadIdx.x; i < cnt * a.n3; i += blockDim.x) gt[i] = a.dG[base * a.n3 + i];
        for (int i = threadIdx.x; i < cnt * K1; i += blockDim.x) {
            int j = i / K1, kk = i % K1;
            float v = 1.0f;
            if (kk < a.K) {
                size_t e = base + j;
                if (!a.shifted) v = a.V[e * a.K + kk];
                else {
                    int t = (int)(e % a.T);
                    v = (t == 0) ? a.y0[(e / a.T) * a.K + kk] : a.V[(e - 1) * a.K + kk];
                }
            }
            vt[i] = v;
        }
        __syncthreads();
        if (valid)
            for (int j = 0; j < cnt; ++j) acc = fmaf(gt[j * a.n3 + g], vt[j * K1 + k], acc);
        __syncthreads();
    }
    if (valid) a.partial[(size_t)blockIdx.x * outs + o] = acc;
}

// Stage 1 for small gates (n3 <= 32, K <= 8): lane g keeps out[g][0..K] in registers; the warps of
// CTA p take blocks of four consecutive positions of slice p in turn (warp w: blocks w, w + 8, ...),
// a lane reading its dG[e][g] (one coalesced row per position) and the row V[e][:] (broadcast).
// The eight warp sums are added in warp order, so the result is bit-reproducible.
__global__ void __launch_bounds__(256) wgrad_small_kernel(WgradArgs a)
{
    constexpr int KMAX = 8, WARPS = 8, BLK = 4;
    __shared__ float part[WARPS][32 * (KMAX + 1)];
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    const int K = a.K, K1 = K + 1, n3 = a.n3;
    const size_t e0 = (size_t)blockIdx.x * a.slice;
    const size_t e1 = min(a.N, e0 + a.slice);
    const bool vec = (K % 4 == 0) && ((((uintptr_t)a.V | (uintptr_t)a.y0) & 15) == 0);
    float acc[KMAX + 1];
#pragma unroll
    for (int k = 0; k <= KMAX; ++k) acc[k] = 0.0f;
    for (size_t base = e0 + (size_t)warp * BLK; base < e1; base += (size_t)WARPS * BLK) {
        float dg[BLK], v[BLK][KMAX];
        size_t seq = 0;
        int t = 0;                                        // (seq, t) of position base + u, carried along
        if (a.shifted) { seq = base / (size_t)a.T; t = (int)(base - seq * (size_t)a.T); }
#pragma unroll
        for (int u = 0; u < BLK; ++u) {
            const size_t e = base + u;
            const bool in = e < e1;
            dg[u] = (in && lane < n3) ? a.dG[e * n3 + lane] : 0.0f;
            const float *row = a.V;                       // row of V paired with position e
            if (in) {
                if (!a.shifted) row = a.V + e * K;
                else row = (t == 0) ? a.y0 + seq * K : a.V + (e - 1) * K;
            }
            if (++t >= a.T) { t = 0; ++seq; }
            if (vec) {
#pragma unroll
                for (int q = 0; q < KMAX / 4; ++q) {
                    float4 f = make_float4(0.0f, 0.0f, 0.0f, 0.0f);
                    if (in && 4 * q < K) f = __ldg(reinterpret_cast<const float4 *>(row) + q);
                    v[u][4 * q] = f.x; v[u][4 * q + 1] = f.y; v[u][4 * q + 2] = f.z; v[u][4 * q + 3] = f.w;
                }
            } else {
#pragma unroll
                for (int k = 0; k < KMAX; ++k) v[u][k] = (in && k < K) ? __ldg(row + k) : 0.0f;
            }
        }
#pragma unroll
        for (int u = 0; u < BLK; ++u) {
#pragma unroll
            for (int k = 0; k < KMAX; ++k) acc[k] = fmaf(dg[u], v[u][k], acc[k]);
            acc[KMAX] += dg[u];                           // bias column (V = 1)
        }
    }
#pragma unroll
    for (int k = 0; k < KMAX; ++k) part[warp][lane * (KMAX + 1) + k] = acc[k];
    part[warp][lane * (KMAX + 1) + KMAX] = acc[KMAX];
    __syncthreads();
    const int outs = n3 * K1;
    for (int o = threadIdx.x; o < outs; o += blockDim.x) {
        const int g = o / K1, k = o - g * K1;
        const int src = g * (KMAX + 1) + (k < K ? k : KMAX);
        float s = 0.0f;
#pragma unroll
        for (int w = 0; w < WARPS; ++w) s += part[w][src];
        a.partial[(size_t)blockIdx.x * outs + o] = s;
    }
}

// Stage 2: one warp per output.  Lane l adds slices l, l + 32, ... in that order (all loads in
// flight together), then the 32 lane sums are combined by a fixed shuffle tree: the order of the
// additions depends on P only, so the result is bit-reproducible.
__global__ void wgrad_final_kernel(const float *__restrict__ partial, int P, int n3, int K,
                                   float *__restrict__ dW, float *__restrict__ db)
{
    const int K1 = K + 1, outs = n3 * K1;
    const int o = (blockIdx.x * blockDim.x + threadIdx.x) >> 5, lane = threadIdx.x & 31;
    if (o >= outs) return;
    float acc = 0.0f;
#pragma unroll 4
    for (int p = lane; p < P; p += 32) acc += partial[(size_t)p * outs + o];
#pragma unroll
    for (int d = 16; d > 0; d >>= 1) acc += __shfl_down_sync(0xffffffffu, acc, d);
    if (lane == 0) {
        const int g = o / K1, k = o % K1;
        if (k < K) dW[(size_t)g * K + k] = acc;
        else db[g] = acc;
    }
}

// ------------------------------------------------------------------ a9: classifier glue
// partial mean-pool: grid (segments, B), block = n threads
__global__ void pool_partial_kernel(const float *__restrict__ y, int T, int n, int seg_len,
                                    float *__restrict__ partial /*[B][S][n]*/)
{
    const int sgm = blockIdx.x, S = gridDim.x;
    const size_t seq = blockIdx.y;
    const int t0 = sgm * seg_len, t1 = min(T, t0 + seg_len);
    const int i = threadIdx.x;
    float acc = 0.0f;
    for (int t = t0; t < t1; ++t) acc += y[(seq * T + t) * n + i];
    partial[(seq * S + sgm) * n + i] = acc;
}

// head: pooled mean, logits, softmax cross-entropy (mean over batch), gradients of the head,
// gradient w.r.t. the pooled vector scaled by 1/T.  One CTA, thread-serial where order matters.
__global__ void head_kernel(const float *__restrict__ pool_partial, int S, int B, int T, int n,
                            int ncls, const float *__restrict__ W_o, const float *__restrict__ b_o,
                            const int *__restrict__ labels, float *__restrict__ pooled /*[B][n]*/,
                            float *__restrict__ dlog /*[B][ncls]*/, float *__restrict__ gpool /*[B][n]*/,
                            float *__restrict__ dW_o, float *__restrict__ db_o,
                            float *__restrict__ loss_out)
{
    for (int idx = threadIdx.x; idx < B * n; idx += blockDim.x) {
        int seq = idx / n, i = idx % n;
        float acc = 0.0f;
        for (int s = 0; s < S; ++s) acc += pool_partial[((size_t)seq * S + s) * n + i];
        pooled[idx] = acc / (float)T;
    }
    __syncthreads();
    for (int idx = threadIdx.x; idx < B * ncls; idx += blockDim.x) {
        int seq = idx / ncls, c = idx % ncls;
        float l = b_o[c];
        for (int i = 0; i < n; ++i) l = fmaf(W_o[c * n + i], pooled[seq * n + i], l);
        dlog[idx] = l;
    }
    __syncthreads();
    __shared__ float s_loss;
    if (threadIdx.x == 0) {
        float loss = 0.0f;
        for (int seq = 0; seq < B; ++seq) {
            float *l = dlog + seq * ncls;
            float mx = l[0];
            for (int c = 1; c < ncls; ++c) mx = fmaxf(mx, l[c]);
            float se = 0.0f;
            for (int c = 0; c < ncls; ++c) se += expf(l[c] - mx);
            float lse = mx + logf(se);
            loss += lse - l[labels[seq]];
            for (int c = 0; c < ncls; ++c)
                l[c] = (expf(l[c] - lse) - (c == labels[seq] ? 1.0f : 0.0f)) / (float)B;
        }
        s_loss = loss / (float)B;
        *loss_out = s_loss;
    }
    __syncthreads();
    for (int idx = threadIdx.x; idx < ncls * n; idx += blockDim.x) {
        int c = idx / n, i = idx % n;
        float acc = 0.0f;
        for (int seq = 0; seq < B; ++seq) acc = fmaf(dlog[seq * ncls + c], pooled[seq * n + i], acc);
        dW_o[idx] = acc;
    }
    for (int c = threadIdx.x; c < ncls; c += blockDim.x) {
        float acc = 0.0f;
        for (int seq = 0; seq < B; ++seq) acc += dlog[seq * ncls + c];
        db_o[c] = acc;
    }
    for (int idx = threadIdx.x; idx < B * n; idx += blockDim.x) {
        int seq = idx / n, i = idx % n;
        float acc = 0.0f;
        for (int c = 0; c < ncls; ++c) acc = fmaf(W_o[c * n + i], dlog[seq * ncls + c], acc);
        gpool[idx] = acc / (float)T;
    }
}

// gy[b][t][i] = gpool[b][i] for every t
__global__ void broadcast_gy_kernel(const float *__restrict__ gpool, float *__restrict__ gy,
                                    size_t total, int T, int n)
{
    size_t idx = (size_t)blockIdx.x * blockDim.x + threadIdx.x;
    if (idx >= total) return;
    size_t seq = idx / ((size_t)T * n);
    int i = (int)(idx % n);
    gy[idx] = gpool[seq * n + i];
}


// ------------------------------------------------------------------ forward-mode derivative of the cell (Sec. 3.1.1)
// df at every position for a direction (dW_i, dW_h, db_i, db_h, dx) at fixed h = y_prev:
//   da_r = du_r + dW_hr h + db_hr,  da_z likewise,  dq = dW_hn h + db_hn,  du = x dW_i^T + db_i + dx W_i^T (precomputed)
//   dr = r (1-r) da_r,  dz = z (1-z) da_z,  dc = (1-c^2)(du_n + dr q + r dq),  df = (1-z) dc + (h-c) dz
// One thread per (position, row); W_h and dW_h in shared memory (rows padded by one float).
struct JvpArgs {
    const float *W_h, *b_h, *dW_h, *db_h;    // dW_h, db_h may be nullptr (= 0)
    const float *u;                          // [B,T,3n]  x W_i^T + b_i
    const float *du1, *du2;                  // [B,T,3n]  x dW_i^T + db_i  and  dx W_i^T (either may be nullptr)
    const float *y, *y0;
    float *df;                               // [B,T,n] out
    int B, T, n;
};

__global__ void jvp_cell_kernel(JvpArgs a)
{
    extern __shared__ float sW[];
    const int n = a.n, ld = n + 1;
    float *sD = sW + 3 * n * ld;
    float *sb = sD + 3 * n * ld, *sdb = sb + 3 * n;
    for (int i = threadIdx.x; i < 3 * n * n; i += blockDim.x) {
        sW[(i / n) * ld + (i % n)] = a.W_h[i];
        sD[(i / n) * ld + (i % n)] = a.dW_h ? a.dW_h[i] : 0.0f;
    }
    for (int i = threadIdx.x; i < 3 * n; i += blockDim.x) { sb[i] = a.b_h[i]; sdb[i] = a.db_h ? a.db_h[i] : 0.0f; }
    __syncthreads();
    const int epb = blockDim.x / n;
    const int le = threadIdx.x / n, i = threadIdx.x % n;
    const size_t N = (size_t)a.B * a.T;
    for (size_t e = (size_t)blockIdx.x * epb + le; le < epb && e < N; e += (size_t)gridDim.x * epb) {
        const int t = (int)(e % a.T);
        const size_t seq = e / a.T;
        const float *hp = (t == 0) ? a.y0 + seq * n : a.y + (e - 1) * n;
        float gr = sb[i], gz = sb[n + i], gq = sb[2 * n + i];
        float dar = sdb[i], daz = sdb[n + i], dq = sdb[2 * n + i];
        for (int k = 0; k < n; ++k) {
            const float h = hp[k];
            gr = fmaf(sW[i * ld + k], h, gr);
            gz = fmaf(sW[(n + i) * ld + k], h, gz);
            gq = fmaf(sW[(2 * n + i) * ld + k], h, gq);
            dar = fmaf(sD[i * ld + k], h, dar);
            daz = fmaf(sD[(n + i) * ld + k], h, daz);
            dq = fmaf(sD[(2 * n + i) * ld + k], h, dq);
        }
        const float *ue = a.u + e * 3 * n;
        float dun = 0.0f;
        if (a.du1) { const float *d = a.du1 + e * 3 * n; dar += d[i]; daz += d[n + i]; dun += d[2 * n + i]; }
        if (a.du2) { const float *d = a.du2 + e * 3 * n; dar += d[i]; daz += d[n + i]; dun += d[2 * n + i]; }
        const float r = sigmoidf_acc(ue[i] + gr);
        const float z = sigmoidf_acc(ue[n + i] + gz);
        const float c = tanhf(ue[2 * n + i] + r * gq);
        const float dr = r * (1.0f - r) * dar;
        const float dz = z * (1.0f - z) * daz;
        const float dc = (1.0f - c * c) * (dun + dr * gq + r * dq);
        a.df[e * n + i] = (1.0f - z) * dc + (hp[i] - c) * dz;
    }
}

// ---------------------------------------------------------------- a second cell: LSTM (Sec. 3.4: any f behind the same iteration)
// State s = [h; c] of 2k components, gates (i, f, g, o):  c' = f c + i g,  h' = o tanh(c'),  f(s, x) = [h'; c'].
// One thread per (position, unit): the unit's four pre-activations from W_h in shared memory and the projected input
// u = x W_i^T + b, then its two rows of the closed-form state Jacobian (rows h'_u and c'_u; columns h then c)
//   dc'/dh = c f(1-f) W_hf + g i(1-i) W_hi + i(1-g^2) W_hg,   dc'/dc = f,
//   dh'/dh = tanh(c') o(1-o) W_ho + o(1 - tanh^2 c') dc'/dh,  dh'/dc = o(1 - tanh^2 c') f
// and rhs = f - J s_prev (Eq. 3).
struct LstmCellArgs {
    const float *W_h;    // [4k,k]
    const float *u;      // [B,T,4k]
    const float *s;      // [B,T,2k] current guess
    const float *s0;     // [B,2k]
    float *J;            // [B,T,2k,2k]
    float *rhs;          // [B,T,2k]
    int B, T, k;
    const StatusBlock *st;
};

__global__ void lstm_cell_kernel(LstmCellArgs a)
{
    if (loop_ended(a.st)) return;
    extern __shared__ float sWl[];
    const int k = a.k, ld = k + 1, n = 2 * k;
    for (int i = threadIdx.x; i < 4 * k * k; i += blockDim.x) sWl[(i / k) * ld + (i % k)] = a.W_h[i];
    __syncthreads();
    const int epb = blockDim.x / k;
    const int le = threadIdx.x / k, un = threadIdx.x % k;
    const size_t N = (size_t)a.B * a.T;
    for (size_t e = (size_t)blockIdx.x * epb + le; le < epb && e < N; e += (size_t)gridDim.x * epb) {
        const int t = (int)(e % a.T);
        const size_t seq = e / a.T;
        const float *sp = (t == 0) ? a.s0 + seq * n : a.s + (e - 1) * n;
        const float *ue = a.u + e * 4 * k;
        float ai = ue[un], af = ue[k + un], ag = ue[2 * k + un], ao = ue[3 * k + un];
        for (int j = 0; j < k; ++j) {
            const float h = sp[j];
            ai = fmaf(sWl[un * ld + j], h, ai);
            af = fmaf(sWl[(k + un) * ld + j], h, af);
            ag = fmaf(sWl[(2 * k + un) * ld + j], h, ag);
            ao = fmaf(sWl[(3 * k + un) * ld + j], h, ao);
        }
        const float gi = sigmoidf_acc(ai), gf = sigmoidf_acc(af), gg = tanhf(ag), go = sigmoidf_acc(ao);
        const float c = sp[k + un];
        const float cn = fmaf(gf, c, gi * gg);
        const float tc = tanhf(cn);
        const float hn = go * tc;
        const float dti = gg * gi * (1.0f - gi), dtf = c * gf * (1.0f - gf), dtg = gi * (1.0f - gg * gg);
        const float dho = tc * go * (1.0f - go), dhc = go * (1.0f - tc * tc);
        float *Jh = a.J + (e * n + un) * n, *Jc = a.J + (e * n + k + un) * n;
        float jh_s = dhc * gf * c, jc_s = gf * c;                  // (J s_prev) of the two rows: the diagonal c-parts first
        for (int j = 0; j < k; ++j) {
            const float dcdh = fmaf(dti, sWl[un * ld + j], fmaf(dtf, sWl[(k + un) * ld + j], dtg * sWl[(2 * k + un) * ld + j]));
            const float dhdh = fmaf(dho, sWl[(3 * k + un) * ld + j], dhc * dcdh);
            Jc[j] = dcdh; Jh[j] = dhdh;
            Jc[k + j] = (j == un) ? gf : 0.0f;
            Jh[k + j] = (j == un) ? dhc * gf : 0.0f;
            jc_s = fmaf(dcdh, sp[j], jc_s);
            jh_s = fmaf(dhdh, sp[j], jh_s);
        }
        a.rhs[e * n + un] = hn - jh_s;
        a.rhs[e * n + k + un] = cn - jc_s;
    }
}

// ---------------------------------------------------------------- ODE instantiation of L_G^{-1} (Sec. 3.3)
// dy/dt + G(t) y = z(t) with G, z constant at their mid-point values on every interval [t_k, t_{k+1}]:
//     y_{k+1} = Gbar_k y_k + zbar_k,   Gbar_k = exp(-G_k D_k),   zbar_k = G_k^{-1} (I - Gbar_k) z_k,
// both read off ONE exponential of the augmented (n+1) x (n+1) matrix [[-G_k D_k, z_k D_k], [0, 0]] =
// [[Gbar_k, zbar_k], [0, 1]] (no inverse: singular G is fine).  One thread per interval: scaling and squaring with a
// degree-9 Taylor polynomial (norm <= 1/4 after scaling: truncation 3e-13), the three work matrices in shared memory
// laid out [element][thread] (conflict-free).  Writes the scan's inputs: J[b][k+1] = Gbar_k, rhs[b][k+1] = zbar_k,
// and J[b][0] = I, rhs[b][0] = 0, so that the forward scan from y0 returns y[b][0] = y0.
constexpr int ODE_THREADS = 64;
constexpr int ODE_MAX_N = 8;

__global__ void __launch_bounds__(ODE_THREADS) ode_discretise_kernel(const float *__restrict__ G, const float *__restrict__ z,
                                                                     const float *__restrict__ t, float *__restrict__ J,
                                                                     float *__restrict__ rhs, int B, int T, int n)
{
    extern __shared__ float sm_ode[];
    const int m = n + 1, mm = m * m, tid = threadIdx.x;
    float *A = sm_ode, *P = A + mm * ODE_THREADS, *Q = P + mm * ODE_THREADS;
#define AT(M_, i_, j_) M_[((i_) * m + (j_)) * ODE_THREADS + tid]
    const size_t total = (size_t)B * T;
    for (size_t e = (size_t)blockIdx.x * ODE_THREADS + tid; e < total; e += (size_t)gridDim.x * ODE_THREADS) {
        const int k = (int)(e % T);                    // this thread writes position k of its sequence
        float *Jo = J + e * n * n, *ro = rhs + e * n;
        if (k == 0) {
            for (int i = 0; i < n; ++i) {
                ro[i] = 0.0f;
                for (int j = 0; j < n; ++j) Jo[i * n + j] = (i == j) ? 1.0f : 0.0f;
            }
            continue;
        }
        const float D = t[k] - t[k - 1];
        const float *G0 = G + (e - 1) * n * n, *G1 = G + e * n * n, *z0 = z + (e - 1) * n, *z1 = z + e * n;
        float norm = 0.0f;
        for (int i = 0; i < m; ++i) {
            float rs = 0.0f;
            for (int j = 0; j < m; ++j) {
                float v = 0.0f;
                if (i < n) v = (j < n) ? -0.5f * (G0[i * n + j] + G1[i * n + j]) * D : 0.5f * (z0[i] + z1[i]) * D;
                AT(A, i, j) = v;
                rs += fabsf(v);
            }
            norm = fmaxf(norm, rs);
        }
        int s = 0;
        float scale = 1.0f;
        while (norm * scale > 0.25f && s < 60) { scale *= 0.5f; ++s; }
        if (!(norm <= 3.0e38f)) s = 0;                 // non-finite input: let it propagate
        for (int i = 0; i < m; ++i)
            for (int j = 0; j < m; ++j) { AT(A, i, j) *= scale; AT(P, i, j) = (i == j) ? 1.0f : 0.0f; }
        for (int kk = 9; kk >= 1; --kk) {              // Horner: P <- I + (A P) / kk
            const float inv = 1.0f / (float)kk;
            for (int i = 0; i < m; ++i)
                for (int j = 0; j < m; ++j) {
                    float acc = 0.0f;
                    for (int l = 0; l < m; ++l) acc = fmaf(AT(A, i, l), AT(P, l, j), acc);
                    AT(Q, i, j) = fmaf(acc, inv, (i == j) ? 1.0f : 0.0f);
                }
            for (int i = 0; i < m; ++i)
                for (int j = 0; j < m; ++j) AT(P, i, j) = AT(Q, i, j);
        }
        for (int q = 0; q < s; ++q) {                  // undo the scaling: square s times
            for (int i = 0; i < m; ++i)
                for (int j = 0; j < m; ++j) {
                    float acc = 0.0f;
                    for (int l = 0; l < m; ++l) acc = fmaf(AT(P, i, l), AT(P, l, j), acc);
                    AT(Q, i, j) = acc;
                }
            for (int i = 0; i < m; ++i)
                for (int j = 0; j < m; ++j) AT(P, i, j) = AT(Q, i, j);
        }
        for (int i = 0; i < n; ++i) {
            for (int j = 0; j < n; ++j) Jo[i * n + j] = AT(P, i, j);
            ro[i] = AT(P, i, n);
        }
    }
#undef AT
}

// ---------------------------------------------------------------- multi-head GRU: strided views <-> dense batches
// A head of stride s over [B,T] is s interleaved sequences per batch entry (Sec. 4.4): sequence (b, p) holds the
// positions t = p + s t', t' = 0 .. T'-1 with T' = ceil(T / s); shorter phases are padded at the END with zeros
// (a GRU is causal: padding behind the last position changes nothing before it).
//   pack  : dst[(b s + p), t', c] = src[b, p + s t', off + c]     (src rows of C_src channels; 0 past T)
//   unpack: dst[b, p + s t', off + c] (+)= src[(b s + p), t', c]  (valid positions only)
// V = 4: channels moved as 128-bit words (C, the row strides, off and the pointers multiples of 4 floats / 16 bytes).
template <int V>
__global__ void mh_pack_kernel(const float *__restrict__ src, float *__restrict__ dst, int B, int T, int s, int Tp, int C,
                               int C_src, int off)
{
    const int Cv = C / V;
    const size_t total = (size_t)B * s * Tp * Cv;
    for (size_t i = (size_t)blockIdx.x * blockDim.x + threadIdx.x; i < total; i += (size_t)gridDim.x * blockDim.x) {
        const int c = (int)(i % Cv) * V;
        const size_t r = i / Cv;
        const int tp = (int)(r % Tp);
        const size_t q = r / Tp;
        const int p = (int)(q % s);
        const size_t b = q / s;
        const long long t = (long long)p + (long long)s * tp;
        if constexpr (V == 4) {
            float4 v = make_float4(0.0f, 0.0f, 0.0f, 0.0f);
            if (t < T) v = *reinterpret_cast<const float4 *>(src + (b * T + (size_t)t) * C_src + off + c);
            *reinterpret_cast<float4 *>(dst + r * C + c) = v;
        } else {
            dst[r * C + c] = t < T ? src[(b * T + (size_t)t) * C_src + off + c] : 0.0f;
        }
    }
}

template <int V>
__global__ void mh_unpack_kernel(const float *__restrict__ src, float *__restrict__ dst, int B, int T, int s, int Tp, int C,
                                 int C_dst, int off, int accumulate)
{
    const int Cv = C / V;
    const size_t total = (size_t)B * s * Tp * Cv;
    for (size_t i = (size_t)blockIdx.x * blockDim.x + threadIdx.x; i < total; i += (size_t)gridDim.x * blockDim.x) {
        const int c = (int)(i % Cv) * V;
        const size_t r = i / Cv;
        const int tp = (int)(r % Tp);
        const size_t q = r / Tp;
        const int p = (int)(q % s);
        const size_t b = q / s;
        const long long t = (long long)p + (long long)s * tp;
        if (t < T) {
            float *d = dst + (b * T + (size_t)t) * C_dst + off + c;
            if constexpr (V == 4) {
                float4 v = *reinterpret_cast<const float4 *>(src + r * C + c);
                if (accumulate) {
                    const float4 o = *reinterpret_cast<const float4 *>(d);
                    v = make_float4(o.x + v.x, o.y + v.y, o.z + v.z, o.w + v.w);
                }
                *reinterpret_cast<float4 *>(d) = v;
            } else {
                *d = accumulate ? *d + src[r * C + c] : src[r * C + c];
            }
        }
    }
}

// y0s[(b s + p), i] = y0[b, h, i]
__global__ void mh_y0_pack_kernel(const float *__restrict__ y0, float *__restrict__ y0s, int B, int s, int n, int H, int h)
{
    const size_t total = (size_t)B * s * n;
    for (size_t i = (size_t)blockIdx.x * blockDim.x + threadIdx.x; i < total; i += (size_t)gridDim.x * blockDim.x) {
        const int c = (int)(i % n);
        const size_t b = i / n / s;
        y0s[i] = y0[(b * H + h) * n + c];
    }
}

// dy0[b, h, i] = sum over the phases p, in order, of dy0s[(b s + p), i]
__global__ void mh_dy0_reduce_kernel(const float *__restrict__ dy0s, float *__restrict__ dy0, int B, int s, int n, int H, int h)
{
    const size_t total = (size_t)B * n;
    for (size_t i = (size_t)blockIdx.x * blockDim.x + threadIdx.x; i < total; i += (size_t)gridDim.x * blockDim.x) {
        const int c = (int)(i % n);
        const size_t b = i / n;
        float acc = 0.0f;
        for (int p = 0; p < s; ++p) acc += dy0s[(b * s + p) * n + c];
        dy0[(b * H + h) * n + c] = acc;
    }
}

}  // namespace deer
