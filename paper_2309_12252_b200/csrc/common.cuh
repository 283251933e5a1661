// Shared definitions of the DEER-GRU CUDA library (device structs, launch bookkeeping).
#pragma once
#include <cuda_runtime.h>
#include <stdint.h>
#include <atomic>
#include "../../include/deer.h"

namespace deer {

extern std::atomic<long long> g_launches;
void set_error(cudaError_t e, const char *where);

#define DEER_CHECK_LAUNCH(where)                                   \
    do {                                                           \
        ::deer::g_launches.fetch_add(1);                           \
        cudaError_t e_ = cudaGetLastError();                       \
        if (e_ != cudaSuccess) {                                   \
            ::deer::set_error(e_, where);                          \
            return DEER_ERR_CUDA;                                  \
        }                                                          \
    } while (0)

// Optional per-kernel timing (CUDA events on the launching stream) for benchmarks.
struct KernelScope {
    const char *name;
    cudaStream_t st;
    cudaEvent_t e0 = nullptr, e1 = nullptr;
    KernelScope(const char *name, cudaStream_t st);
    ~KernelScope();
};

// Launch statement wrapped with bookkeeping:  DEER_KERNEL("name", stream, kernel<<<...>>>(args));
#define DEER_KERNEL(kname, stream, ...)                            \
    do {                                                           \
        {                                                          \
            ::deer::KernelScope ks_(kname, stream);                \
            __VA_ARGS__;                                           \
        }                                                          \
        DEER_CHECK_LAUNCH(kname);                                  \
    } while (0)

// Launch with the programmatic-stream-serialization attribute (see pdl_prologue) when `overlap`:
//   DEER_KERNEL_PDL("name", overlap, stream, kernel, grid, block, smem, args...)
// Measured: the overlap pays for the small-n kernels (config 2: -4 %, config 1: -12 %) and costs for
// n >= 16 at small T (CTAs of two kernels with different shared-memory footprints resident together:
// n = 64, T = 1000: 2.1 ms with, 1.5 ms without), so only the n <= 8 kernels ask for it.
template <typename... KArgs, typename... Args>
static inline cudaError_t launch_pdl(bool overlap, void (*kern)(KArgs...), unsigned grid, unsigned block, size_t smem, cudaStream_t st,
                                     Args... args)
{
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3(grid); cfg.blockDim = dim3(block); cfg.dynamicSmemBytes = smem; cfg.stream = st;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = overlap ? 1 : 0;
    cfg.attrs = attr; cfg.numAttrs = 1;
    return cudaLaunchKernelEx(&cfg, kern, KArgs(args)...);
}

#define DEER_KERNEL_PDL(kname, overlap, stream, kern, grid, block, smem, ...)               \
    do {                                                                                    \
        {                                                                                   \
            ::deer::KernelScope ks_(kname, stream);                                         \
            ::deer::launch_pdl(overlap, kern, grid, block, smem, stream, __VA_ARGS__);      \
        }                                                                                   \
        DEER_CHECK_LAUNCH(kname);                                                           \
    } while (0)

#define DEER_CHECK_CUDA(call, where)                               \
    do {                                                           \
        cudaError_t e_ = (call);                                   \
        if (e_ != cudaSuccess) {                                   \
            ::deer::set_error(e_, where);                          \
            return DEER_ERR_CUDA;                                  \
        }                                                          \
    } while (0)

// Device-resident status of one evaluation (first 256 bytes of the workspace).
struct StatusBlock {
    unsigned err_bits;   // max |y_new - y| of the running body, as the bits of a non-negative float
    unsigned flags;      // FLAG_* bits raised by kernels
    int iters;           // bodies executed so far (device-side loop control)
    int done;            // 1 once the loop condition failed
    unsigned tile_counter;  // dynamic tile id for the single-pass scan (n >= 16 kernels)
    unsigned role_counter;  // role tickets of the single-pass scan (first ones: resolvers); the n <= 8
                            // kernels take their tile ids from it too (ticket - resolvers)
    unsigned err_last_bits; // err of the last executed body
    unsigned exit_counter;  // CTAs of the running single-pass scan that have finished
    int ctl_mode;        // 1: the last CTA of a single-pass scan takes the Newton loop decision
    int max_iter;
    float tol;
    unsigned pad0;
    float *trace;        // err after each body (first ERR_TRACE_CAP bodies), or nullptr
    unsigned pad[50];
};
static_assert(sizeof(StatusBlock) == 256, "status block is one 256-byte line");
constexpr int ERR_TRACE_CAP = 1024;

constexpr unsigned FLAG_NONFINITE = 1u;
constexpr unsigned FLAG_TIMEOUT = 2u;

// One linear-recurrence problem in "scan order".  Position s = 0..T-1 of the
// scan corresponds to t = s (forward) or t = T-1-s (reverse); the matrix of
// position s is J[t] (forward) or J[t+1]^T (reverse; identity at s = 0).
struct ScanArgs {
    const float *J;      // [B,T,n,n]
    const float *b;      // [B,T,n]
    const float *y0;     // [B,n] or nullptr
    float *y;            // [B,T,n] out
    const float *yold;   // [B,T,n] or nullptr: previous iterate for max|y - yold|
    int B, T, n, reverse;
    int L, nch;          // chunk length, chunks per sequence
    float *carA;         // [B,nch,n,n] chunk aggregates (matrix part)
    float *carB;         // [B,nch,n]   chunk aggregates (vector part)
    float *starts;       // [B,nch,n]   state entering each chunk
    StatusBlock *st;
    const float *Wh;     // [3n,n] hidden weights when J holds coefficient rows [B,T,n,4] instead of
                         // matrices (the scan generates J_t itself); nullptr otherwise
    int residual;        // 1: Newton-update form (App. A.1): b holds f - y_old, the scan solves for the
                         // update d_t = J_t d_{t-1} + b_t from d_{-1} = 0 and writes y = y_old + d, err = max|d|
    unsigned spin_limit; // polls a bounded wait makes before it gives up (0: the default, SPIN_LIMIT)
    int no_resolve;      // 1: resolver CTAs return at once, so every wait for an entering state runs
                         // out (DEER_FLAG_EXPIRE_WAITS; exercises the timeout path, nothing else)
};

struct CellArgs {
    const float *W_h;    // [3n,n]
    const float *b_h;    // [3n]
    const float *u;      // [B,T,3n] input projection  x W_i^T + b_i  (nullptr: project on the fly from x)
    const float *x;      // [B,T,m]  only read when u == nullptr
    const float *W_i;    // [3n,m]
    const float *b_i;    // [3n]
    int m;
    const float *y;      // [B,T,n] current trajectory guess
    const float *y0;     // [B,n]
    float *J;            // [B,T,n,n] out
    float *rhs;          // [B,T,n]   out: f - J y_prev   (nullptr: skip)
    int B, T, n;
    const StatusBlock *st;   // nullptr, or: skip all work once st->done is set (Newton loop ended)
    int coef_only;           // wide kernels: write the coefficient rows {k_r, a_z, k_n, z} [B,T,n,4] to J
                             // instead of the matrices (the scan generates J_t from them)
    int residual;            // coefficient-row kernels: rhs receives the residual f - y[t] of the Newton-update
                             // form (App. A.1) instead of f - J y_prev
};

// Programmatic dependent launch: a kernel of the Newton loop lets the next launch in the stream be set
// up and its CTAs become resident as soon as all of this kernel's CTAs are running, then waits for the
// previous kernel to have completed (with its memory visible) before it reads anything that kernel
// produced.  Without the launch attribute both instructions do nothing.
__device__ __forceinline__ void pdl_prologue()
{
    asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
    asm volatile("griddepcontrol.wait;" ::: "memory");
}

// Device-side loop control lets the host enqueue Newton bodies ahead of knowing whether they
// are needed: every kernel of a body returns at once when the loop has already ended.
__device__ __forceinline__ bool loop_ended(const StatusBlock *st)
{
    return st != nullptr && *(volatile const int *)&st->done != 0;
}

// End of one Newton body (App. B.1 loop): record err, count the body, decide whether the loop goes on
// (err > tol and fewer than max_iter bodies).  A NaN err fails "err > tol" and ends the loop, as in
// the listing; an infinite err ends it too.  Single thread.
__device__ __forceinline__ void newton_decide(StatusBlock *st, float tol, int max_iter, float *trace)
{
    const unsigned bits = *(volatile unsigned *)&st->err_bits;
    const float e = __uint_as_float(bits);
    const int k = st->iters;
    if (trace && k < ERR_TRACE_CAP) trace[k] = e;
    st->iters = k + 1;
    st->err_last_bits = bits;
    st->err_bits = 0u;
    if (!(e > tol) || !(e <= 3.402823466e38f) || k + 1 >= max_iter) st->done = 1;
}

// Called by one thread of every CTA of a single-pass scan after the CTA's last global write.  The
// last CTA to leave rewinds the per-launch counters (the launch leaves its flag and state words
// cleared as well: every word is cleared by its only reader) and, in loop-control mode, takes the
// Newton decision, so a body needs no separate control or clearing launch.
// decide = false: a launch that is not the last one of its scan (counters are rewound, no decision).
__device__ __forceinline__ void scan_epilogue(StatusBlock *st, bool decide = true)
{
    __threadfence();
    const unsigned prev = atomicAdd(&st->exit_counter, 1u);
    if (prev + 1u != gridDim.x) return;
    __threadfence();
    st->exit_counter = 0u;
    st->tile_counter = 0u;
    st->role_counter = 0u;
    if (decide && st->ctl_mode) newton_decide(st, st->tol, st->max_iter, st->trace);
}

// Is flat position e = seq * T + t the first of its sequence?  (32-bit division whenever e fits.)
__device__ __forceinline__ bool seq_start(size_t e, int T, size_t &seq)
{
    if (e <= 0xffffffffull) {
        const unsigned q = (unsigned)e / (unsigned)T;
        seq = q;
        return (unsigned)e - q * (unsigned)T == 0u;
    }
    seq = e / (size_t)T;
    return e - seq * (size_t)T == 0;
}

__device__ __forceinline__ float sigmoidf_acc(float a) { return 1.0f / (1.0f + expf(-a)); }

// Gate activations for the issue-bound small-n cell kernel: ex2.approx / rcp.approx based (a few
// instructions instead of ~25 each).  exp2 and the reciprocal are good to 2 ulp and the product
// a*log2(e) adds |a| * 6e-8 relative to the exponential, so sigma is within 3e-7 and tanh within
// 2e-7 ABSOLUTE of the exact value on the whole real line (saturated ends included; NaN stays NaN)
// -- three orders of magnitude below the 1e-4 tolerance the evaluation is solved and checked to.
__device__ __forceinline__ float sigmoidf_gate(float a) { return __fdividef(1.0f, 1.0f + __expf(-a)); }
__device__ __forceinline__ float tanhf_gate(float a)
{
    const float e = __expf(-2.0f * fabsf(a));            // in (0, 1]
    return copysignf(__fdividef(1.0f - e, 1.0f + e), a);
}

// Packed pairs of fp32 operations (sm_100: one instruction for two lanes of a 64-bit register pair).
__device__ __forceinline__ float2 ffma2(float2 a, float2 b, float2 c)
{
    unsigned long long ra, rb, rc, rd;
    asm("mov.b64 %0, {%1, %2};" : "=l"(ra) : "f"(a.x), "f"(a.y));
    asm("mov.b64 %0, {%1, %2};" : "=l"(rb) : "f"(b.x), "f"(b.y));
    asm("mov.b64 %0, {%1, %2};" : "=l"(rc) : "f"(c.x), "f"(c.y));
    asm("fma.rn.f32x2 %0, %1, %2, %3;" : "=l"(rd) : "l"(ra), "l"(rb), "l"(rc));
    float2 d;
    asm("mov.b64 {%0, %1}, %2;" : "=f"(d.x), "=f"(d.y) : "l"(rd));
    return d;
}
__device__ __forceinline__ float2 fmul2(float2 a, float2 b)
{
    unsigned long long ra, rb, rd;
    asm("mov.b64 %0, {%1, %2};" : "=l"(ra) : "f"(a.x), "f"(a.y));
    asm("mov.b64 %0, {%1, %2};" : "=l"(rb) : "f"(b.x), "f"(b.y));
    asm("mul.rn.f32x2 %0, %1, %2;" : "=l"(rd) : "l"(ra), "l"(rb));
    float2 d;
    asm("mov.b64 {%0, %1}, %2;" : "=f"(d.x), "=f"(d.y) : "l"(rd));
    return d;
}

__device__ __forceinline__ float2 fadd2(float2 a, float2 b)
{
    unsigned long long ra, rb, rd;
    asm("mov.b64 %0, {%1, %2};" : "=l"(ra) : "f"(a.x), "f"(a.y));
    asm("mov.b64 %0, {%1, %2};" : "=l"(rb) : "f"(b.x), "f"(b.y));
    asm("add.rn.f32x2 %0, %1, %2;" : "=l"(rd) : "l"(ra), "l"(rb));
    float2 d;
    asm("mov.b64 {%0, %1}, %2;" : "=f"(d.x), "=f"(d.y) : "l"(rd));
    return d;
}
__device__ __forceinline__ float ex2_approx(float x) { float y; asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x)); return y; }
__device__ __forceinline__ float rcp_approx(float x) { float y; asm("rcp.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x)); return y; }

// The gate activations on a pair of values: the arithmetic around the two special-function-unit results (the scaling of
// the exponent, 1 +- e, the final product) runs as packed f32x2 instructions; same approximate units as the scalar forms.
__device__ __forceinline__ float2 sigmoid2_gate(float2 a)
{
    const float2 t = fmul2(a, make_float2(-1.4426950408889634f, -1.4426950408889634f));
    const float2 d = fadd2(make_float2(ex2_approx(t.x), ex2_approx(t.y)), make_float2(1.0f, 1.0f));
    return make_float2(rcp_approx(d.x), rcp_approx(d.y));
}
__device__ __forceinline__ float2 tanh2_gate(float2 a)
{
    const float2 t = fmul2(make_float2(fabsf(a.x), fabsf(a.y)), make_float2(-2.8853900817779268f, -2.8853900817779268f));
    const float2 e = make_float2(ex2_approx(t.x), ex2_approx(t.y));                     // exp(-2 |a|) in (0, 1]
    const float2 one = make_float2(1.0f, 1.0f);
    const float2 num = ffma2(e, make_float2(-1.0f, -1.0f), one), den = fadd2(e, one);
    const float2 q = fmul2(num, make_float2(rcp_approx(den.x), rcp_approx(den.y)));
    return make_float2(copysignf(q.x, a.x), copysignf(q.y, a.y));
}

__device__ __forceinline__ unsigned absdiff_bits(float a, float b) {
    return __float_as_uint(fabsf(a - b));   // NaN keeps bits above +inf: an integer max propagates it
}

// 256-bit global store (sm_100): one request per 32 contiguous bytes of a lane; the address must be 32-byte aligned
__device__ __forceinline__ void st_global_v8(float *p, const float4 &a, const float4 &b)
{
    asm volatile("st.global.v8.f32 [%0], {%1, %2, %3, %4, %5, %6, %7, %8};" ::"l"(p), "f"(a.x), "f"(a.y), "f"(a.z), "f"(a.w),
                 "f"(b.x), "f"(b.y), "f"(b.z), "f"(b.w)
                 : "memory");
}

static inline size_t align_up(size_t v, size_t a = 256) { return (v + a - 1) / a * a; }

}  // namespace deer
