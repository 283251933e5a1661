/*
 * deer.h -- C ABI of the DEER-GRU hot path for NVIDIA B200 (sm_100a).
 *
 * DEER evaluates a non-linear recurrence y_t = f(y_{t-1}, x_t) for all t at
 * once by a Newton-type fixed-point iteration (Sec. 3.1, Eq. 3 with Eq. 5);
 * each iteration evaluates the cell f and its n x n state Jacobian at every
 * position of the current guess, forms the right-hand side and solves the
 * linear recurrence y_t = J_t y_{t-1} + b_t with an associative scan
 * (Sec. 3.3-3.4, Eq. 9-10).  The cell here is a GRU (Sec. 4.1).
 *
 * General rules for every entry point
 *   - All array arguments are DEVICE pointers owned by the caller, fp32,
 *     dense row-major with the shapes stated, unless marked "host".
 *   - The library never allocates or frees device memory: scratch comes from
 *     the caller-supplied workspace `ws` of at least deer_workspace_bytes()
 *     bytes, 256-byte aligned.  The workspace contents are undefined on entry
 *     and on return; two calls that overlap in time need distinct workspaces.
 *   - `stream` is a cudaStream_t passed as void* (NULL = the legacy default
 *     stream).  Work is enqueued on it; deer_gru_eval synchronises the stream
 *     before it returns because it writes host outputs, the others do not
 *     unless stated.
 *   - Return value: a deer_status.  >= 0 are outcomes of a run that executed,
 *     < 0 mean nothing (or nothing useful) was computed.  Nothing aborts,
 *     throws or traps.  Every device-side wait is bounded: when one expires
 *     the kernels drain and raise a flag in the workspace's status block.
 *     The entry points that synchronise (deer_gru_eval*, deer_gru_classifier_step)
 *     return DEER_ERR_DEVICE_TIMEOUT themselves; the asynchronous ones
 *     (deer_linrec_scan*, deer_gru_vjp) return before the kernels have run, so
 *     their caller asks with deer_workspace_status / deer_noalloc_status.
 *   - Batch index b, position t, 0-based.  y[b][-1] = y0[b].
 *   - Supported hidden sizes: 1 <= n <= 64 (tuned kernels for n in
 *     {1, 2, 4, 8, 16, 32, 64}, a generic kernel for the rest); 1 <= m <= 1024.
 */
#ifndef DEER_H_
#define DEER_H_

#include <stddef.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef enum deer_status {
    DEER_OK = 0,
    DEER_NOT_CONVERGED = 1,        /* max_iter bodies ran, err still > tol; y = last iterate */
    DEER_NONFINITE = 2,            /* NaN/Inf appeared in the iterate; y = last iterate */
    DEER_ERR_INVALID_ARG = -1,     /* NULL pointer, non-positive size, NaN tol, max_iter < 1 ... */
    DEER_ERR_UNSUPPORTED_N = -2,   /* n or m outside the supported range */
    DEER_ERR_WORKSPACE = -3,       /* ws NULL, misaligned or smaller than deer_workspace_bytes() */
    DEER_ERR_CUDA = -4,            /* a CUDA runtime call failed; see deer_last_error() */
    DEER_ERR_DEVICE_TIMEOUT = -5   /* a bounded device-side wait expired; outputs are invalid */
} deer_status;

/* GRU parameters (Sec. 4.1 uses a standard GRU; the paper prints no
 * equations, the cell evaluated is
 *     r = sigmoid(W_ir x + b_ir + W_hr h + b_hr)
 *     z = sigmoid(W_iz x + b_iz + W_hz h + b_hz)
 *     c = tanh   (W_in x + b_in + r * (W_hn h + b_hn))
 *     f(h, x) = (1 - z) * c + z * h ).
 * Packed along the leading axis in gate order (r, z, n). */
typedef struct deer_gru_params {
    int n;              /* hidden size */
    int m;              /* input size  */
    const float *W_i;   /* [3n, m] */
    const float *W_h;   /* [3n, n] */
    const float *b_i;   /* [3n]    */
    const float *b_h;   /* [3n]    */
} deer_gru_params;

/* Parameter gradients, same shapes as the parameters; overwritten. */
typedef struct deer_gru_grads {
    float *dW_i, *dW_h, *db_i, *db_h;
} deer_gru_grads;

/* Operations for deer_workspace_bytes(). */
enum { DEER_OP_EVAL = 0, DEER_OP_SCAN = 1, DEER_OP_VJP = 2, DEER_OP_CLASSIFIER = 3, DEER_OP_ODE = 4,
       DEER_OP_LSTM = 5 /* n = the number of LSTM units k */ };

/* Flags (bit-or). */
enum {
    DEER_FLAG_WARM_START = 1,   /* deer_gru_eval: y holds the initial guess on entry (Sec. 3.1:
                                   the previous training step's solution may seed the next) */
    DEER_FLAG_GENERIC    = 2,   /* force the generic (any-n) kernels; for testing */
    DEER_FLAG_MATERIALIZE = 4,  /* deer_gru_eval, n = 16, 32 and 64: have the cell write the Jacobians
                                   J [B,T,n,n] to the workspace and scan them, instead of writing
                                   four coefficient vectors per position from which the scan builds
                                   J_t itself (the default there; the two agree to rounding) */
    DEER_FLAG_TCGEN05    = 8,   /* n = 64 scans: run the chain product (Eq. 10's matrix half) as
                                   tcgen05.mma in tensor memory instead of register-resident
                                   mma.sync fragments; same results to rounding, currently slower */
    DEER_FLAG_EXPIRE_WAITS = 16, /* test aid for the bounded waits of the single-pass scans: the
                                   CTAs that publish the states entering each tile return at once
                                   and every wait gives up after a few polls, so the scan drains
                                   and the call reports DEER_ERR_DEVICE_TIMEOUT (outputs invalid).
                                   Nothing traps or hangs; the workspace can be used again */
    DEER_FLAG_COEF_ROWS  = 32   /* deer_gru_cell_jac, n = 16, 32 and 64: write the four coefficient
                                   vectors per position instead of the matrices (see there) */
};

/* Bytes of workspace needed by `op` at the given sizes (0 if the sizes are
 * invalid).  m is ignored for DEER_OP_SCAN.  The tile length of the scan, and
 * with it the size, depends on the SM count of the current device: query with
 * the device current on which the call will run. */
size_t deer_workspace_bytes(int op, int B, int T, int n, int m, int flags);

/* Solve the linear recurrence (the operator L_G^{-1} of Eq. 10 with J = -G)
 * with a chunked associative scan whose combine is
 * (A2, b2) o (A1, b1) = (A2 A1, A2 b1 + b2)  (Eq. 9):
 *   reverse == 0 :  y[b][t] = J[b][t] y[b][t-1] + b[b][t],   y[b][-1] = y0[b]
 *   reverse != 0 :  y[b][t] = b[b][t] + J[b][t+1]^T y[b][t+1],
 *                   y[b][T-1] = b[b][T-1] + y0[b]
 *     (the adjoint of the forward solve with respect to b -- the "dual
 *      operator" of Sec. 3.1.1; J[b][0] is not read).
 *   J  [B,T,n,n]  row = output component        b  [B,T,n]
 *   y0 [B,n] or NULL (= zeros)                  y  [B,T,n] out (must not alias J or b)
 * Asynchronous on `stream`: the return value covers argument checks and launches
 * only; deer_workspace_status(ws, stream) tells whether the kernels ran to the end.
 * Returns DEER_OK or a negative status. */
int deer_linrec_scan(const float *J, const float *b, const float *y0, int B, int T, int n,
                     int reverse, float *y, void *ws, size_t ws_bytes, int flags, void *stream);

/* The same scan for callers that cannot hand the library a workspace.
 * (No counterpart in the paper: this exists for integration, not for the method.)
 * Some hosts of this library may not allocate device memory at the point where
 * they need a scan: code that runs inside a framework's memory-planned region,
 * a real-time loop that must not touch the allocator, or a plug-in that is only
 * given its input and output buffers.  For them this variant takes its scratch
 * from a fixed array that is part of the library image: DEER_NOALLOC_SCRATCH_BYTES
 * of device memory, reserved on every GPU that loads the library for as long as
 * the process lives.  It calls no cudaMalloc / cudaFree and no allocating
 * routine of any other library.
 *   - Arguments, layouts and results are those of deer_linrec_scan.
 *   - Sizes whose scratch (deer_workspace_bytes(DEER_OP_SCAN, ...)) exceeds
 *     DEER_NOALLOC_SCRATCH_BYTES are refused with DEER_ERR_WORKSPACE and a
 *     message in deer_last_error(); nothing runs.
 *   - The first call on each device looks up the array's device address (with
 *     that device current); make that first call outside any stream capture.
 *   - All calls on a device share the one array, which keeps whatever the last
 *     call left in it; the entry point clears the words that must start at zero
 *     itself.  Two calls that overlap on the GPU (different streams, no ordering
 *     between them) would race on the array: order them.
 * Asynchronous on `stream` (deer_noalloc_status tells whether the kernels ran to
 * the end).  Returns DEER_OK or a negative status. */
#define DEER_NOALLOC_SCRATCH_BYTES (8u << 20)
int deer_linrec_scan_noalloc(const float *J, const float *b, const float *y0, int B, int T, int n,
                             int reverse, float *y, void *stream);

/* Outcome of the last asynchronous call (deer_linrec_scan, deer_gru_vjp) that used
 * workspace `ws`: synchronises `stream`, reads the status block at the head of the
 * workspace and returns DEER_OK, or DEER_ERR_DEVICE_TIMEOUT when a bounded wait of
 * that call's kernels expired (its outputs are then invalid).  No counterpart in the
 * paper: failure reporting of this implementation's scan (Eq. 9-10). */
int deer_workspace_status(const void *ws, void *stream);

/* The same for the last deer_linrec_scan_noalloc call on the current device. */
int deer_noalloc_status(void *stream);

/* Launch geometry the scan (Eq. 9-10: chunked, chunk aggregates combined, applied back
 * down) would use for these sizes on the current device, for tests and tuning:
 *   out[0] 1: single-pass kernels, 0: three-kernel (reduce / carry / apply) path
 *          (taken for other n, DEER_FLAG_GENERIC, unaligned buffers -- not visible
 *          here -- and batches too large for the single-pass resolvers)
 *   out[1] positions per tile (chunk)      out[2] positions per warp chain where the
 *          kernel chooses it at launch (n = 8, 16, 32), else 0
 *   out[3] tiles per sequence              out[4] resolver CTAs (single-pass)
 *   out[5] SM count the choice was made for
 * `out` is a host array of 6 ints.  Returns DEER_OK or a negative status. */
int deer_scan_geometry(int B, int T, int n, int flags, int *out);

/* The steps of one Newton body before the solve, on their own (Eq. 3 with Eq. 5;
 * App. B.1: function evaluation, Jacobian, rhs): at every position of the guess y,
 * with y_prev[b][t] = t ? y[b][t-1] : y0[b],
 *     J[b][t]   = df/dy_prev (y_prev, x[b][t])            [B,T,n,n] out, row = output
 *     rhs[b][t] = f(y_prev, x[b][t]) - J[b][t] y_prev     [B,T,n]   out
 * by the kernel deer_gru_eval uses for these sizes (DEER_FLAG_GENERIC: the any-n kernel).
 * With DEER_FLAG_COEF_ROWS (n = 16, 32, 64, 16-byte aligned buffers) J receives instead the
 * coefficient rows [B,T,n,4] = {k_r, a_z, k_n, z} from which the scans of deer_gru_eval
 * build J = diag(k_r) W_hr + diag(a_z) W_hz + diag(k_n) W_hn + diag(z) themselves.
 *   ws : workspace of deer_workspace_bytes(DEER_OP_EVAL, ...) bytes (holds x W_i^T + b_i)
 * Asynchronous on `stream`.  Returns DEER_OK or a negative status. */
int deer_gru_cell_jac(const deer_gru_params *params, const float *x, const float *y0, const float *y,
                      int B, int T, float *J, float *rhs, void *ws, size_t ws_bytes, int flags,
                      void *stream);

/* Evaluate the GRU over whole sequences with the DEER iteration (Eq. 3 with
 * G = -df/dy, Eq. 5; loop of App. B.1): starting from y = 0 (or the guess in
 * y when DEER_FLAG_WARM_START), repeat { J, f at the shifted guess;
 * rhs = f - J y_prev; y_new = scan(J, rhs, y0); err = max |y_new - y| } while
 * err > tol and fewer than max_iter bodies have run (err starts at 1e10).
 * One global err over the whole batch.
 *   x [B,T,m]   y0 [B,n]   y [B,T,n] out (in: guess if warm start)
 *   tol        : paper default 1e-4 for fp32; a negative tol runs exactly
 *                max_iter bodies; NaN is invalid
 *   iters      : host out, number of executed bodies (may be NULL)
 *   err        : host out, last max |y_new - y|       (may be NULL)
 *   err_trace  : host out [max_iter], err after each body, rest untouched (may be NULL)
 * Synchronises `stream`.  Returns DEER_OK, DEER_NOT_CONVERGED, DEER_NONFINITE
 * or a negative status. */
int deer_gru_eval(const deer_gru_params *params, const float *x, const float *y0, int B, int T,
                  float tol, int max_iter, float *y, int *iters, float *err, float *err_trace,
                  void *ws, size_t ws_bytes, int flags, void *stream);

/* deer_gru_eval with diagnostics of the last executed body (App. B.1: the
 * quantity the loop tests is max |y_new - y|):
 *   err_b      : host out [B], max |y_new - y| per sequence (may be NULL)
 *   err_argmax : host out, flat index (b*T + t)*n + i of the element where the
 *                global maximum is attained; ties go to the smallest index
 *                (may be NULL)
 * Both are pure functions of the last two iterates and, like iters, err and
 * every bit of y, identical across runs.  T*n must fit 32 bits.  Everything
 * else as deer_gru_eval. */
int deer_gru_eval_diag(const deer_gru_params *params, const float *x, const float *y0, int B, int T,
                       float tol, int max_iter, float *y, int *iters, float *err, float *err_trace,
                       float *err_b, unsigned long long *err_argmax, void *ws, size_t ws_bytes, int flags,
                       void *stream);

/* deer_gru_eval with the sequence data in HOST memory (the end-to-end call):
 * copies x_host to x_dev, evaluates into y_dev as deer_gru_eval does, copies
 * the result to y_host (asynchronously when the host buffers are page-locked).
 * A batch that deer_gru_eval_host_chunks(B, T, ...) splits is evaluated
 * chunk by chunk, each chunk with its own Newton loop (sequences
 * are independent: the batch is a map over sequences, Sec. 3), so that on
 * copy streams owned by the library chunk c + 1 arrives and chunk c - 1
 * leaves while chunk c is evaluated; each chunk's result is exactly what
 * deer_gru_eval returns for those sequences alone, `iters` and `err` are the
 * largest over the chunks, the status is the worst.  A batch of one chunk runs
 * copy, bodies and copy on `stream`, the result copy enqueued behind the first
 * group of bodies.
 *   x_host [B,T,m] host in     y_host [B,T,n] host out
 *   x_dev  [B,T,m], y_dev [B,T,n] : device staging buffers owned by the caller
 *            (y_dev holds the guess on entry if DEER_FLAG_WARM_START, and the
 *            result on return)
 *   params, y0, ws : device, as for deer_gru_eval (ws sized for the whole B)
 * Work already enqueued on `stream` is waited for before the first copy; the
 * call synchronises `stream` and its copy streams, and calls on one device
 * are serialised.  Returns what deer_gru_eval returns. */
int deer_gru_eval_host(const deer_gru_params *params, const float *x_host, const float *y0, int B, int T,
                       float tol, int max_iter, float *y_host, int *iters, float *err, float *x_dev,
                       float *y_dev, void *ws, size_t ws_bytes, int flags, void *stream);

/* The chunks of deer_gru_eval_host for a batch of B sequences of length T:
 * returns their number nc (1 when the batch is not split, at most
 * DEER_HOST_MAX_CHUNKS; 0 for invalid sizes) and, when `first` is not NULL
 * (host, room for DEER_HOST_MAX_CHUNKS + 1 entries), writes the first
 * sequence of every chunk and B itself to first[0 .. nc].  Chunks hold about
 * 2^19 positions; from three chunks on the first and the last are about half
 * as long as the others, because their copies are the two that no evaluation
 * hides.  deer_gru_eval_host_chunk returns the largest chunk's sequence
 * count.  Host only. */
#define DEER_HOST_MAX_CHUNKS 8
int deer_gru_eval_host_chunks(int B, int T, int *first);
int deer_gru_eval_host_chunk(int B, int T);

/* Gradient through the evaluated sequence (Eq. 7): given gy = dL/dy at a
 * trajectory y, lambda = gy L_G^{-1} by ONE reverse scan with the Jacobians
 * recomputed at y (Sec. 3.1.1 allows saving or recomputing them), then the
 * cell's vector-Jacobian product at every position, summed over positions in
 * a fixed order (bit-reproducible).
 *   y  [B,T,n] trajectory (normally deer_gru_eval's output)   gy [B,T,n]
 *   dparams : device arrays, overwritten       dx  [B,T,m] or NULL
 *   dy0 [B,n] or NULL
 * Asynchronous on `stream` (see deer_workspace_status).  Returns DEER_OK or a
 * negative status. */
int deer_gru_vjp(const deer_gru_params *params, const float *x, const float *y0, const float *y,
                 const float *gy, int B, int T, const deer_gru_grads *dparams, float *dx,
                 float *dy0, void *ws, size_t ws_bytes, int flags, void *stream);

/* Forward-mode derivative (Sec. 3.1.1, the forward derivative equation): the first-order change dy of the
 * trajectory y under a change of the parameters, the inputs and the initial state,
 *     dy = L_G^{-1}[ (df/dtheta) dtheta + (df/dx) dx ]   started from dy0,
 * by ONE forward scan with the Jacobians at y (the same operator the iteration inverts; Eq. 9-10):
 * df at every position from the direction, then dy[t] = J[t] dy[t-1] + df[t], dy[-1] = dy0.
 *   params  : the parameters          dparams : the direction in parameter space, same n and m; device
 *             arrays W_i with b_i and/or W_h with b_h may be NULL pairs (= 0); dparams itself may be NULL
 *   x [B,T,m]   dx [B,T,m] or NULL    y0 [B,n]   dy0 [B,n] or NULL    y [B,T,n] the trajectory
 *   dy [B,T,n] out          ws : deer_workspace_bytes(DEER_OP_VJP, ...) bytes
 * Asynchronous on `stream` (see deer_workspace_status).  Returns DEER_OK or a negative status. */
int deer_gru_jvp(const deer_gru_params *params, const deer_gru_params *dparams, const float *x, const float *dx,
                 const float *y0, const float *dy0, const float *y, int B, int T, float *dy, void *ws,
                 size_t ws_bytes, int flags, void *stream);

/* A second cell behind the same iteration (Sec. 3.4: the method applies to any y_i = f(y_{i-1}, x_i, theta); Eq. 3
 * with Eq. 5): an LSTM with k units, state s = [h; c] of 2k components, gates in the order (i, f, g, o),
 *     a = W_i x + b + W_h h,  c' = sigmoid(a_f) c + sigmoid(a_i) tanh(a_g),  h' = sigmoid(a_o) tanh(c'),
 * evaluated over whole sequences exactly as deer_gru_eval evaluates the GRU: cell + closed-form 2k x 2k state
 * Jacobian + rhs at every position (one kernel), the scan kernels of deer_linrec_scan at state size 2k, the same
 * device-side loop control.  (Forward evaluation only; no tuned cell kernel.) */
typedef struct deer_lstm_params {
    int k;              /* units; the state has 2k components, 2k <= 64 */
    int m;              /* input size */
    const float *W_i;   /* [4k, m] */
    const float *W_h;   /* [4k, k] */
    const float *b;     /* [4k]    */
} deer_lstm_params;

/*   x [B,T,m]   s0 [B,2k]   s [B,T,2k] out (the guess on entry if DEER_FLAG_WARM_START)
 *   iters, err : host out (may be NULL)     ws : deer_workspace_bytes(DEER_OP_LSTM, B, T, k, m, 0) bytes
 * Synchronises `stream`.  Returns DEER_OK, DEER_NOT_CONVERGED, DEER_NONFINITE or a negative status. */
int deer_lstm_eval(const deer_lstm_params *params, const float *x, const float *s0, int B, int T, float tol,
                   int max_iter, float *s, int *iters, float *err, void *ws, size_t ws_bytes, int flags,
                   void *stream);

/* The linear operator L_G^{-1} of an ordinary differential equation (Sec. 3.3): solve
 *     dy/dt + G(t) y = z(t),   y(t_0) = y0
 * on the time points t_0 < ... < t_{T-1}, with G and z taken constant at their MID-POINT values on every interval
 * (third-order local truncation error, App. A.5):
 *     y_{k+1} = Gbar_k y_k + zbar_k,   Gbar_k = exp(-G_k D_k),   zbar_k = G_k^{-1} (I - Gbar_k) z_k,
 *     G_k = (G(t_k) + G(t_{k+1})) / 2,  z_k likewise,  D_k = t_{k+1} - t_k
 * -- a batched small matrix exponential per interval (of the augmented matrix [[-G_k D_k, z_k D_k], [0, 0]], which
 * yields Gbar_k and zbar_k together and needs no inverse), then the same associative scan as the discrete case (Eq. 9).
 * This is the operator a DEER iteration for an ODE applies once per body (the caller evaluates f and its Jacobian).
 *   G [B,T,n,n]   z [B,T,n]   t [T] (device, increasing)   y0 [B,n]   y [B,T,n] out, y[b][0] = y0[b]
 *   n <= 8 (DEER_ERR_UNSUPPORTED_N above);  ws : deer_workspace_bytes(DEER_OP_ODE, B, T, n, 0, 0) bytes
 * Asynchronous on `stream` (see deer_workspace_status).  Returns DEER_OK or a negative status. */
int deer_ode_linear_solve(const float *G, const float *z, const float *t, const float *y0, int B, int T, int n,
                          float *y, void *ws, size_t ws_bytes, int flags, void *stream);

/* One training step of the long-series classifier (App. B.3 shapes: mean
 * over the sequence, then a linear decoder and cross-entropy): two stacked
 * GRU layers of equal hidden size n (layer 1 reads x [B,T,m], layer 2 reads
 * layer 1's states), zero initial states, p = mean_t y2, logits = W_o p + b_o,
 * loss = mean over the batch of softmax cross-entropy; forward by
 * deer_gru_eval per layer, backward by deer_gru_vjp per layer.
 *   W_o [n_classes, n]  b_o [n_classes]  labels [B] int32 (device)
 *   loss : host out      iters : host out [2] (may be NULL)
 *   g1, g2 : parameter gradients per layer;  dW_o [n_classes,n], db_o [n_classes] device out
 * Synchronises `stream`.  Returns the worst status of the two evaluations, or
 * DEER_ERR_DEVICE_TIMEOUT when a bounded wait expired in either backward pass. */
int deer_gru_classifier_step(const deer_gru_params *layer1, const deer_gru_params *layer2,
                             const float *W_o, const float *b_o, int n_classes, const float *x,
                             const int *labels, int B, int T, float tol, int max_iter,
                             float *loss, int *iters, const deer_gru_grads *g1,
                             const deer_gru_grads *g2, float *dW_o, float *db_o, void *ws,
                             size_t ws_bytes, int flags, void *stream);

/* Multi-head GRU unit (Sec. 4.4 "Sequence classification with multiple heads RNN"; App. B.4): H independent
 * GRU heads of hidden size n, every one reading the whole input x[b][t] (m channels) with its own
 * parameters, head h advancing with stride s_h,
 *     y[b][t][h] = f_h(y[b][t - s_h][h], x[b][t]),      y[b][t'][h] = y0[b][h] for t' < 0,
 * so that a head of stride s is s interleaved sequences.  The Jacobian of the whole unit is block-diagonal
 * over the heads (the paper's way around the n^3 cost of the scan): every head is evaluated by the DEER
 * iteration of deer_gru_eval on its own, its interleaved sequences laid out as a dense batch of B * s_h
 * sequences of ceil(T / s_h) positions by a gather kernel (heads of equal stride share the gathered input).
 *   heads   : HOST array of H parameter sets (device pointers inside), equal n and m
 *   strides : HOST array of H strides >= 1 (the paper uses 2^0 ... 2^7, assigned uniformly to 32 heads)
 *   x [B,T,m]   y0 [B,H,n]   y [B,T,H,n] out (the heads' states side by side; the guess on entry if
 *   DEER_FLAG_WARM_START)      iters : host out [H], bodies executed per head (may be NULL)
 *   ws : deer_multihead_workspace_bytes(...) bytes
 * Synchronises `stream`.  Returns the worst status of the heads' evaluations or a negative status. */
size_t deer_multihead_workspace_bytes(const int *strides, int H, int B, int T, int n, int m, int flags);
int deer_gru_multihead_eval(const deer_gru_params *heads, const int *strides, int H, const float *x,
                            const float *y0, int B, int T, float tol, int max_iter, float *y, int *iters,
                            void *ws, size_t ws_bytes, int flags, void *stream);

/* Gradient through the multi-head unit (Eq. 7 per head: one reverse scan and the cell's vector-Jacobian
 * product), for dL/dy = gy [B,T,H,n] at the trajectory y:
 *   dheads : HOST array of H gradient sets (device arrays, overwritten)
 *   dx [B,T,m] or NULL : the heads' contributions added head by head in a fixed order
 *   dy0 [B,H,n] or NULL
 * Synchronises `stream`.  Returns DEER_OK, DEER_ERR_DEVICE_TIMEOUT or another negative status. */
int deer_gru_multihead_vjp(const deer_gru_params *heads, const int *strides, int H, const float *x,
                           const float *y0, const float *y, const float *gy, int B, int T,
                           const deer_gru_grads *dheads, float *dx, float *dy0, void *ws, size_t ws_bytes,
                           int flags, void *stream);

/* Text for a status code (static storage). */
const char *deer_status_string(int status);

/* Message of the last CUDA error seen by the calling thread ("" if none). */
const char *deer_last_error(void);

/* Number of kernels this library has launched since it was loaded (all
 * threads); take differences around a region to count its launches. */
long long deer_launch_count(void);

/* Benchmark aid (no counterpart in the paper): while enabled, every kernel
 * launch of the library is bracketed by CUDA events on its stream.
 * deer_profile_read() waits for the recorded events, writes one line
 * "kernel_name launches total_ms" per kernel into buf (NUL-terminated, at
 * most cap bytes), clears the records and returns the full text length.
 * Adds two event records per launch, so it is kept out of timed regions. */
void deer_profile_enable(int on);
size_t deer_profile_read(char *buf, size_t cap);

#ifdef __cplusplus
}
#endif
#endif /* DEER_H_ */
