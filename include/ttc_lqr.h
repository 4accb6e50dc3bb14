/*
 * ttc_lqr.h -- C ABI of the batched finite-horizon LQR solver (the hot path of a
 * Test-Time Control layer), NVIDIA B200 (sm_100a) only.
 *
 * Problem solved, independently for each of N = batch[0]*batch[1]*batch[2] instances
 * (the paper's Eq. 3 / Definition A.1 with time-invariant parameters, written with the
 * usual control indexing):
 *
 *     minimise   sum_{t=0}^{H-1} ( x_t' Q x_t + u_t' R u_t ) + x_H' Q x_H
 *     subject to x_{t+1} = A x_t + B u_t ,  x_0 given
 *
 *     A: n x n,  B: n x m,  Q: n x n symmetric PSD,  R: m x m symmetric PD,  x_0: n.
 *
 * Results (Prop. 3.1 and Alg. 1 of the paper):
 *     P_H = Q ;  for t = H-1..0:
 *         K_t = -(R + B' P_{t+1} B)^{-1} B' P_{t+1} A
 *         P_t = Q + A' P_{t+1} A + (B' P_{t+1} A)' K_t
 *     u_t = K_t x_t ;  x_{t+1} = A x_t + B u_t .
 * Relation to the paper's indexing (h_t = A h_{t-1} + B u_t, t = 1..T, Q_0 = 0):
 * x_t = h_t, u_t = paper's u_{t+1}, K_t = paper's K_{t+1}, P_t = paper's P_t for t >= 1,
 * P_0 = paper's P_0 + Q.  The optimal cost is x_0' P_0 x_0.
 *
 * Two methods compute the same P_t: the sequential Riccati recursion, and a scan over
 * the horizon whose element is the symplectic transition matrix of Thm A.2 stored
 * inverse-free as the triple (A, C = B R^{-1} B', J = Q) (TTC_SCAN).
 *
 * All matrices are row-major and contiguous (leading dimension = number of columns).
 * Instance index i = (i0*batch[1] + i1)*batch[2] + i2; an input operand of instance i
 * starts at element  i0*bstride[0] + i1*bstride[1] + i2*bstride[2]  of its array; a
 * stride of 0 shares the operand along that batch dimension (e.g. per-head A, B, R).
 * Outputs are dense in i.
 *
 * Every function returns a status (0 = TTC_OK, negative = error, nothing enqueued).
 * No function aborts the process; device code never traps and has no unbounded wait.
 */
#ifndef TTC_LQR_H_
#define TTC_LQR_H_

#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

/* status codes */
#define TTC_OK                        0
#define TTC_STATUS_INVALID_ARGUMENT  (-1)
#define TTC_STATUS_CUDA_ERROR        (-2)
#define TTC_STATUS_ALLOC_FAILED      (-3)
#define TTC_STATUS_UNSUPPORTED       (-4)

/* element types of input operands */
#define TTC_F32   0
#define TTC_BF16  1

/* ttc_lqr_config.method */
#define TTC_AUTO     0   /* library picks                                            */
#define TTC_RICCATI  1   /* sequential backward recursion (Prop. 3.1, Alg. 1)        */
#define TTC_SCAN     2   /* symplectic-pair scan over the horizon (Thm A.2 element)  */

/* ttc_lqr_config.math : arithmetic of the n x n contractions */
#define TTC_MATH_AUTO  0  /* FP32 when every input is F32, TF32 when Q or x0 is BF16  */
#define TTC_MATH_FP32  1  /* FFMA, fp32 throughout                                    */
#define TTC_MATH_TF32  2  /* tcgen05 tensor cores, tf32 operands, fp32 accumulate (n = m = 64) */
/* n = m = 64 is served by the tensor-core kernel only with TF32 math (AUTO picks it when Q or x0 is
 * BF16), per-head A, B, R and a time-invariant problem; FP32 math at n = m = 64, and every
 * time-varying / affine / gradient call at n = m = 64, run in the generic one-CTA-per-instance kernel
 * (TTC_KERNEL_RICCATI_CTA), which is one to two orders of magnitude slower. */

/* ttc_lqr_solve flags */
#define TTC_OUT_FIRST_ONLY  1u  /* P is [N][n][n] = P_0 and u is [N][m] = u_0          */
#define TTC_OUT_BF16        2u  /* K, P, x, u are bfloat16 arrays (same shapes), rounded to
                                   nearest even from the float32 results; halves the bytes the
                                   write-bound requests store.  ttc_lqr_solve only, sequential
                                   recursion, n = m in {16, 32, 64 with TF32 math}; other
                                   requests return TTC_STATUS_UNSUPPORTED.  info stays int32. */

/* ttc_lqr_query keys */
#define TTC_QUERY_LAST_LAUNCHES    1  /* kernels launched by the last solve            */
#define TTC_QUERY_WORKSPACE_BYTES  2  /* device bytes currently owned by the handle    */
#define TTC_QUERY_LAST_KERNEL      3  /* id of the main kernel of the last solve       */
#define TTC_QUERY_TOTAL_LAUNCHES   4  /* kernels launched since create                 */
#define TTC_QUERY_DEVICE_ERROR     5  /* 0, or non-zero if a bounded wait inside the last
                                         kernel ran out (synchronises the device)       */

/* ids returned by TTC_QUERY_LAST_KERNEL */
#define TTC_KERNEL_NONE           0
#define TTC_KERNEL_RICCATI_CTA    1  /* generic: one CTA per instance, FFMA            */
#define TTC_KERNEL_RICCATI_WARP   2  /* register-tiled FFMA, several instances per CTA */
#define TTC_KERNEL_SCAN           4  /* symplectic-pair scan + gain/rollout kernel     */
#define TTC_KERNEL_RICCATI_UMMA   5  /* tcgen05 contractions (tensor memory), n = m = 64 */
#define TTC_KERNEL_LAYER          6  /* contextualised layer: parameters synthesised in-kernel */
#define TTC_KERNEL_SIGMA_BASELINE 7 /* baseline: row-normalised reverse symplectic product   */

typedef struct ttc_lqr_handle ttc_lqr_handle; /* opaque; owned by the library */

/* One input operand.  `ptr` is owned by the caller and only read.  For ttc_lqr_solve it
 * is a DEVICE pointer (on the handle's device), for ttc_lqr_solve_host a HOST pointer.
 * It must be aligned to 16 bytes.  Strides are arbitrary non-negative element counts; the
 * fast kernels (tcgen05 for n = m = 64, the fp32 warp kernel for n = m = 16 / 32) read the
 * rows of Q and Qf with 16-byte loads and are chosen only when every batch and time stride
 * of those two operands is a multiple of 16 bytes (4 F32 or 8 BF16 elements); any other
 * stride is served, correctly but much more slowly, by the generic kernel. */
typedef struct {
    const void* ptr;
    int32_t     dtype;       /* TTC_F32 or TTC_BF16 (BF16 only for Q and x0)            */
    int32_t     reserved;    /* set to 0                                                */
    int64_t     bstride[3];  /* element stride per batch dimension; 0 = shared          */
} ttc_operand;

typedef struct {
    int32_t n;               /* state dimension, 1..64                                  */
    int32_t m;               /* control dimension, 1..64                                */
    int32_t max_horizon;     /* largest H that will be passed to solve, >= 1            */
    int32_t device;          /* CUDA device ordinal                                     */
    int64_t batch[3];        /* e.g. {sequences, heads, tokens}; each >= 1              */
    int32_t method;          /* TTC_AUTO | TTC_RICCATI | TTC_SCAN                       */
    int32_t math;            /* TTC_MATH_*                                              */
} ttc_lqr_config;

/*
 * Create a solver for a fixed problem shape (the paper's problem statement, Eq. 3 and
 * Definition A.1, fixes what a "problem" is: {A,B,Q,R}, h_0 and a horizon).
 * Validates cfg, selects the device, returns an opaque handle in *out.  The handle owns
 * only its device workspace, which is allocated on first need inside a solve call (such
 * a call synchronises the device once) and freed by ttc_lqr_destroy.
 * Errors: INVALID_ARGUMENT (null pointers, sizes out of range), UNSUPPORTED (method/math
 * not available for this shape), CUDA_ERROR (no such device / not an sm_100 device).
 */
int ttc_lqr_create(const ttc_lqr_config* cfg, ttc_lqr_handle** out);

/*
 * Solve all N instances (Prop. 3.1 / Alg. 1; or the symplectic scan built on Thm A.2's
 * transition matrices when the method is TTC_SCAN).  Asynchronous: kernels are enqueued
 * on `cuda_stream` (a cudaStream_t; NULL = the default stream) and the call returns;
 * outputs are valid once the stream reaches that point.  One handle serves one stream at
 * a time.
 *
 * Inputs (device):  A [n][n], B [n][m], R [m][m] as F32;  Q [n][n], x0 [n] as F32 or BF16.
 *                   x0 may be NULL when neither x nor u is requested.
 * Outputs (device, F32 -- BF16 with TTC_OUT_BF16 --, written completely, each may be NULL = not wanted):
 *     K    [N][H][m][n]
 *     P    [N][H+1][n][n]    (or [N][n][n] = P_0   with TTC_OUT_FIRST_ONLY)
 *     x    [N][H+1][n]
 *     u    [N][H][m]         (or [N][m]    = u_0   with TTC_OUT_FIRST_ONLY)
 *     info [N] int32: 0 = solved; t*m + j + 1 > 0 = pivot j (0-based) of R + B'P_{t+1}B at
 *          time index t was not positive (R not positive definite, Q indefinite, or NaN
 *          input).  All requested outputs of such an instance are filled with quiet NaN;
 *          other instances are unaffected.
 * Output pointers must be 16-byte aligned.
 * Errors: INVALID_ARGUMENT (null handle/operand, H < 1 or H > max_horizon, bad dtype,
 * misaligned pointer), ALLOC_FAILED (workspace), CUDA_ERROR (launch failure).
 */
int ttc_lqr_solve(ttc_lqr_handle* h,
                  const ttc_operand* A, const ttc_operand* B, const ttc_operand* Q,
                  const ttc_operand* R, const ttc_operand* x0, int32_t H,
                  float* K, float* P, float* x, float* u, int32_t* info,
                  uint32_t flags, void* cuda_stream);

/*
 * ttc_lqr_solve with the state cost handed over in factored form (Parameterization paragraph of the TTC-Net
 * section: Q is a combination of a few basis directions plus a diagonal):
 *     Q = scale * U U' + diag(d),      U [n][rank] and d [n] per instance (F32 or BF16, batch strides as any operand),
 *     1 <= rank <= n, scale >= 0.  Q is symmetric positive semi-definite by construction when d >= 0.
 * The library expands Q on the device into a float32 workspace it owns (N n^2 floats, one more kernel launch) and then
 * runs exactly the ttc_lqr_solve path on it; the caller stores and transfers n (rank + 1) numbers per instance instead
 * of n^2 (configuration 4: 1.2 KB instead of 8 KB).  With TTC_MATH_AUTO the tensor-core path is taken when U is BF16,
 * as for a BF16 dense Q.  Everything else (outputs, info, flags, stream, errors) as ttc_lqr_solve.
 */
int ttc_lqr_solve_lowrank_q(ttc_lqr_handle* h,
                            const ttc_operand* A, const ttc_operand* B, const ttc_operand* U, const ttc_operand* d,
                            int32_t rank, float scale, const ttc_operand* R, const ttc_operand* x0, int32_t H,
                            float* K, float* P, float* x, float* u, int32_t* info,
                            uint32_t flags, void* cuda_stream);

/*
 * Time-varying problem (Definition A.1 / Prop. A.1 with A_t, B_t, Q_t, R_t and a terminal weight Q_f;
 * Alg. 1 with the time indices kept):
 *     minimise   sum_{t=0}^{H-1} ( x_t' Q_t x_t + u_t' R_t u_t ) + x_H' Q_f x_H ,   x_{t+1} = A_t x_t + B_t u_t
 *     P_H = Q_f ;  K_t = -(R_t + B_t' P_{t+1} B_t)^{-1} B_t' P_{t+1} A_t ;  P_t = Q_t + A_t' P_{t+1} A_t + (B_t' P_{t+1} A_t)' K_t .
 * With the paper's h_t = A_t h_{t-1} + B_t u_t (t = 1..T): x_t = h_t, A_t(here) = A_{t+1}(paper), likewise B and R,
 * Q_t(here) = Q_t(paper), Q_f = Q_T.
 * tstride[0..3] are the element strides between consecutive time indices of A, B, Q, R (0 = the same matrix
 * at every t); the matrix of step t of instance i starts at the operand's batch offset + t * tstride.
 * Qf [n][n] (F32 or BF16, batch strides like any operand) is the terminal weight; it may be NULL only when
 * tstride[2] == 0, and then Q_f = Q.  Everything else (outputs, info, flags, stream, errors) as ttc_lqr_solve.
 * Served by the fp32 kernels (n = m = 16 / 32 warp kernel when A, B, R are all shared by the tokens of a head or all
 * per token, generic kernel otherwise); TTC_SCAN handles
 * time-invariant problems only and returns TTC_STATUS_UNSUPPORTED here.
 */
int ttc_lqr_solve_tv(ttc_lqr_handle* h,
                     const ttc_operand* A, const ttc_operand* B, const ttc_operand* Q, const ttc_operand* R,
                     const int64_t tstride[4], const ttc_operand* Qf, const ttc_operand* x0, int32_t H,
                     float* K, float* P, float* x, float* u, int32_t* info,
                     uint32_t flags, void* cuda_stream);

/*
 * Time-varying solve with a LINEAR CONTROL COST (Definition A.1 with r_t; Prop. A.1 / Alg. 1):
 *     stage cost 1/2 (x_t'Q_t x_t + u_t'R_t u_t) + r_t'u_t,   terminal cost 1/2 x_H'Qf x_H
 * (with the linear term the factor 1/2 matters; P_t and K_t are those of ttc_lqr_solve_tv).
 * Value function V_t(x) = 1/2 x'P_t x + p_t'x + c_t, p_H = 0;
 *     k_t = -(R_t + B_t'P_{t+1}B_t)^{-1} (B_t'p_{t+1} + r_t),   p_t = A_t'p_{t+1} + Y'k_t,  Y = B_t'P_{t+1}A_t,
 *     u_t = K_t x_t + k_t,   x_{t+1} = A_t x_t + B_t u_t.
 * In the paper's indexing r_t(here) = r_{t+1}(paper), like A, B and R.  This is the forward solve that the dual
 * problem of Thm 3.2 needs.
 *
 * Arguments as for ttc_lqr_solve_tv, plus: r -- float32 vectors of length m, batch strides as for the
 * other operands, r_tstride = element stride between consecutive time indices (0 = the same vector
 * at every t); kff [N][H][m] receives k_t; pvec receives p_t, [N][H+1][n] or [N][n] = p_0 with
 * TTC_OUT_FIRST_ONLY.  Each output may be NULL.  With TTC_OUT_FIRST_ONLY u = u_0 = K_0 x_0 + k_0.
 * Failed instances: every requested output quiet NaN, info as for ttc_lqr_solve.  The scan method
 * returns TTC_STATUS_UNSUPPORTED.
 */
int ttc_lqr_solve_affine(ttc_lqr_handle* h,
                         const ttc_operand* A, const ttc_operand* B, const ttc_operand* Q, const ttc_operand* R,
                         const int64_t tstride[4], const ttc_operand* Qf,
                         const ttc_operand* r, int64_t r_tstride, const ttc_operand* x0, int32_t H,
                         float* K, float* kff, float* P, float* pvec, float* x, float* u, int32_t* info,
                         uint32_t flags, void* cuda_stream);

/*
 * Gradients of a scalar loss l(o) of the layer output o = u_0* (Thm 3.2: primal and dual LQR), for the
 * time-varying problem of ttc_lqr_solve_tv.  g [N][m] (float32, device) is dl/do.  The call runs
 *   1. the backward Riccati pass (K_t) with the dual problem's linear cost on the first control riding along
 *      (Prop. A.1 with r_0 = g: k_0 = -S_0^{-1} g; every later k_t is zero);
 *   2. both rollouts: x_t, u_t = K_t x_t from x0 (primal), and xd_0 = 0, ud_0 = k_0, ud_t = K_t xd_t (dual);
 *   3. both co-state sequences by  lam_H = Qf x_H,  lam_t = A_t' lam_{t+1} + Q_t x_t;
 *   4. the outer products of the theorem, in this library's time indexing (A_t here = A_{t+1} of the paper):
 *        dA [N][H][n][n]:  lam_{t+1} xd_t' + lamd_{t+1} x_t'      dB [N][H][n][m]:  lam_{t+1} ud_t' + lamd_{t+1} u_t'
 *        dQ [N][H][n][n]:  1/2 (x_t xd_t' + xd_t x_t')            dQf [N][n][n]:    the same at t = H
 *        dR [N][H][m][m]:  1/2 (u_t ud_t' + ud_t u_t')            dx0 [N][n]:       lamd_0
 * and writes the forward output u0 [N][m].  Each output may be NULL (not computed).  Gradients are per instance
 * and per time step: for an operand shared between instances or constant in time the caller sums the slices.
 * dQ, dQf, dR are symmetric (derivatives along symmetric perturbations); Q_t and Qf must be symmetric.
 * All outputs float32, device, 16-byte aligned, row-major; the call is asynchronous on cuda_stream.
 * Failed instances (info != 0): every requested output quiet NaN.  Workspace: K_t, k_t and six vector sequences
 * (N * (H m n + H m + 6 (H+1) max(n, m)) floats), grown on demand.
 * Errors: as ttc_lqr_solve_tv; the scan method returns TTC_STATUS_UNSUPPORTED.
 */
int ttc_lqr_grad(ttc_lqr_handle* h,
                 const ttc_operand* A, const ttc_operand* B, const ttc_operand* Q, const ttc_operand* R,
                 const int64_t tstride[4], const ttc_operand* Qf, const ttc_operand* x0, const float* g, int32_t H,
                 float* dA, float* dB, float* dQ, float* dQf, float* dR, float* dx0, float* u0, int32_t* info,
                 void* cuda_stream);

/*
 * One Test-Time Control layer evaluation per instance with CONTEXTUALISED parameters
 * (Contextualization and Parameterization paragraphs of the TTC-Net section): the LQR parameters
 * of the planning horizon t = 1..T are synthesised inside the kernel from per-instance
 * coefficient vectors and shared basis matrices and are never written to memory:
 *     A_t = I + diag(exp(-t s_gamma_a) .* s_a)                        (diagonal)
 *     B_t = (sum_i s_b[i] B_basis[i]) diag(exp(-t s_gamma_b))
 *     Q_t = diag(exp(-t s_gamma_q)) (sum_i s_q[i] Q_basis[i]) diag(exp(-t s_gamma_q)),  Q_0 = 0,
 *     Q_T = sum_i s_qf[i] Q_basis[i]                                  (terminal override)
 *     R_t = diag(1 / r_inv)                                           (the layer is handed diag(R^-1))
 * for the problem of the LQR section / Definition A.1 without affine terms,
 *     h_t = A_t h_{t-1} + B_t u_t,  cost = sum_{t=1..T} h_t'Q_t h_t + u_t'R_t u_t,
 * solved by the backward recursion of Prop. A.1 / Alg. 1.  Outputs: u1 = u_1* (the layer output,
 * [N][n]) and P0 (the value matrix at t = 0, [N][n][n]: the optimal cost is h0'P0 h0), info [N]
 * (0, or s*n + j + 1 for the first non-positive pivot j of R + B'PB at step s = t - 1; that
 * instance's outputs are quiet NaN).  Each output may be NULL.
 *
 * The handle must have n == m in {16, 32} (else TTC_STATUS_UNSUPPORTED); N is the product of its
 * batch dimensions and instance i of every array is row i.  All pointers are DEVICE memory,
 * float32, dense row-major, 16-byte aligned, owned by the caller and read-only for the call:
 * s_a, s_gamma_a, s_gamma_b, s_gamma_q, r_inv, h0 are [N][n]; s_b, s_q, s_qf are [N][r];
 * B_basis, Q_basis are [r][n][n] (Q_basis[i] symmetric positive semi-definite), 1 <= r <= 64.
 * s_gamma_* >= 0 and r_inv > 0 are the caller's responsibility (softplus outputs in the paper).
 * 1 <= T <= max_horizon of the handle.  Asynchronous on cuda_stream like ttc_lqr_solve.
 */
typedef struct ttc_layer_inputs {
    const float* s_a;
    const float* s_gamma_a;
    const float* s_gamma_b;
    const float* s_gamma_q;
    const float* s_b;
    const float* s_q;
    const float* s_qf;
    const float* r_inv;
    const float* h0;
    const float* B_basis;
    const float* Q_basis;
    int32_t r;
} ttc_layer_inputs;

int ttc_lqr_solve_layer(ttc_lqr_handle* h, const ttc_layer_inputs* in, int32_t T,
                        float* u1, float* P0, int32_t* info, void* cuda_stream);

/*
 * Gradients of a scalar loss l(u_1*) of the contextualised layer's output with respect to everything
 * ttc_lqr_solve_layer is handed (Thm 3.2: primal and dual LQR; then the chain rule through the Contextualization /
 * Parameterization paragraphs).  g [N][n] (device, float32) is dl/du_1*.  The per-step matrices dA_t, dB_t, dQ_t,
 * dR_t of the theorem are never formed: their outer products are reduced as they appear onto
 *     s_a, s_gamma_a, s_gamma_b, s_gamma_q, r_inv, h0   [N][n]         s_b, s_q, s_qf   [N][r]
 * per instance, and onto B_basis, Q_basis [r][n][n], which are shared by all instances and therefore receive the SUM
 * over the instances (accumulated with float atomics: the last bits depend on the order).  The Q_basis gradient is
 * symmetric (derivative along symmetric perturbations, Q_basis[i] being symmetric).  Every member of `out` may be
 * NULL (not computed); u1 (optional) receives the forward output, info as in ttc_lqr_solve_layer.  An instance whose
 * backward pass failed (info != 0) gets quiet NaN in its per-instance gradients and adds nothing to the basis
 * gradients.  All pointers device memory, float32, 16-byte aligned; asynchronous on cuda_stream.
 * Workspace owned by the handle: N (2 T n^2 + (4 T + 5) n) floats, plus 3 N n^2 when a basis gradient is requested.
 * Needs n == m in {16, 32}; 1 <= T <= max_horizon.
 */
typedef struct ttc_layer_grads {
    float* s_a;
    float* s_gamma_a;
    float* s_gamma_b;
    float* s_gamma_q;
    float* s_b;
    float* s_q;
    float* s_qf;
    float* r_inv;
    float* h0;
    float* B_basis;
    float* Q_basis;
} ttc_layer_grads;

int ttc_lqr_layer_grad(ttc_lqr_handle* h, const ttc_layer_inputs* in, int32_t T, const float* g,
                       const ttc_layer_grads* out, float* u1, int32_t* info, void* cuda_stream);

/*
 * BASELINE for comparison, not the recommended solver: the same layer evaluation by the reverse symplectic
 * iteration of Thm 3.3 / Alg. 3 with the row normalisation of the paper's fused kernel (hardware co-design
 * appendix): [Y1 Y2] = [I Q_T] Sigma_T ... Sigma_1 accumulated row by row in registers, each row divided by
 * max(|y1|_1, |y2|_1) after every step, then P0 = Y1^{-1} Y2 by Gauss-Jordan elimination with partial pivoting,
 * lambda_0 = P0 h0, u1 = -R_1^{-1} B_1' A_1^{-T} lambda_0.  Arguments, outputs and errors as ttc_lqr_solve_layer;
 * info is 0 or 1 + the column at which Y1 had no non-zero pivot (outputs quiet NaN).  The product contains
 * A_t^{-1} and propagates [state; co-state] like a shooting method: in float32 its error grows with the horizon
 * (about 1e-5 at T = 2, percent level by T = 16 and no correct digit by T = 32 on the layer16 inputs) where the
 * backward recursion of ttc_lqr_solve_layer stays near 1e-6.  It exists so that the efficiency sweep can time
 * both formulations on the same inputs.
 */
int ttc_lqr_solve_layer_sigma_baseline(ttc_lqr_handle* h, const ttc_layer_inputs* in, int32_t T,
                                       float* u1, float* P0, int32_t* info, void* cuda_stream);

/*
 * ttc_lqr_solve_layer with HOST buffers: every pointer of `in` and u1 / P0 / info are host memory
 * (pinned memory lets the copies run at full speed; pageable memory works).  The call copies the
 * inputs to a device staging buffer owned by the handle, runs the same kernel on an internal
 * stream, copies the requested outputs back and returns after everything has completed
 * (synchronous).  Large batches are cut into up to 32 slices of the instance dimension so that
 * the copy-in of one slice, the solve of the previous one and the copy-out of the one before
 * overlap.  No alignment requirement on host pointers.  Results are identical to
 * ttc_lqr_solve_layer.
 */
int ttc_lqr_solve_layer_host(ttc_lqr_handle* h, const ttc_layer_inputs* in, int32_t T,
                             float* u1, float* P0, int32_t* info);

/*
 * Same computation with HOST buffers (same problem statement as ttc_lqr_solve): operand
 * pointers and all outputs are host memory (pinned memory lets the copies run asynchronously;
 * pageable memory works but serialises them).  The call copies the inputs to device staging
 * buffers owned by the handle, solves on internal streams, copies the requested outputs back
 * and returns after everything has completed (synchronous).  Large problems are cut into up to
 * 32 slices of the last batch dimension so that the copy-in of one slice, the solve of the
 * previous one and the copy-out of the one before overlap; results are identical to
 * ttc_lqr_solve.  Strides have the same meaning.  Flags as for ttc_lqr_solve: with TTC_OUT_BF16
 * K, P, x, u are bfloat16 host arrays, which halves the bytes copied back.
 */
int ttc_lqr_solve_host(ttc_lqr_handle* h,
                       const ttc_operand* A, const ttc_operand* B, const ttc_operand* Q,
                       const ttc_operand* R, const ttc_operand* x0, int32_t H,
                       float* K, float* P, float* x, float* u, int32_t* info,
                       uint32_t flags);

/*
 * Allocation-free variant of the P_0 / u_0 solve.  The paper has no counterpart: this entry
 * point exists for callers that are not allowed to allocate device memory at the moment they
 * need a solve -- code running inside a memory-pool or allocator callback, a plugin whose host
 * framework owns every device allocation, or a real-time loop in which cudaMalloc (which may
 * synchronise the whole device and take an unbounded time) is forbidden.  ttc_lqr_solve cannot
 * serve them because its scan path keeps one value matrix per instance plus a status word in a
 * workspace obtained with cudaMalloc.
 *
 * It computes, with the symplectic-pair scan (method TTC_SCAN, TTC_OUT_FIRST_ONLY), exactly what
 *     ttc_lqr_solve(h, A, B, Q, R, x0, H, NULL, P0, NULL, u0, info, TTC_OUT_FIRST_ONLY, stream)
 * computes on a TTC_SCAN handle of the same shape: P0 [N][n][n], u0 [N][m], info [N] (each may be
 * NULL; x0 may be NULL when u0 is).  No handle is needed.  The scratch (one n x n value matrix and
 * one int32 per instance) lives in a fixed array of TTC_NOALLOC_SCRATCH_BYTES bytes that is part
 * of the library image: every GPU on which the library is loaded holds those bytes until the
 * process exits.  The call makes no cudaMalloc / cudaFree and calls no allocating library
 * routine; the caller still provides every input and output buffer.  Like the other entry
 * points it makes `device` the calling thread's current device (cudaSetDevice).
 *
 * Limits and rules:
 *  - N * (4*n*n) rounded up to 256, plus 4*N, must not exceed TTC_NOALLOC_SCRATCH_BYTES; larger
 *    problems are rejected with TTC_STATUS_INVALID_ARGUMENT and a message naming both numbers
 *    (nothing is enqueued).  Split the batch, or use ttc_lqr_solve.
 *  - The first call on a device looks up the device address of the scratch array (once per
 *    device, with that device current).  Make that first call before starting any stream
 *    capture.
 *  - Every call on a device shares the one array.  Nothing in it has to start at zero (each call
 *    writes every word it later reads) and it keeps the previous call's contents.  Two calls
 *    whose kernels can overlap on the GPU (different streams, or different host threads without
 *    ordering) race on it: order them on one stream or with events.
 * Errors otherwise as for ttc_lqr_solve.
 */
#define TTC_NOALLOC_SCRATCH_BYTES (4u << 20)
int ttc_lqr_solve_first_noalloc(int32_t n, int32_t m, const int64_t batch[3], int32_t device,
                                const ttc_operand* A, const ttc_operand* B, const ttc_operand* Q,
                                const ttc_operand* R, const ttc_operand* x0, int32_t H,
                                float* P0, float* u0, int32_t* info, void* cuda_stream);

/*
 * Self test of the bounded waits (no counterpart in the paper; failure handling of this library): every
 * wait of the tensor-core kernel on an MMA-completion barrier gives up after a fixed number of polls and sets
 * an error word instead of hanging.  This call runs that give-up branch on purpose, safely: a one-warp
 * kernel initialises a barrier on which nothing will ever arrive, polls it `poll_limit` times (1 .. 2^20),
 * and returns by itself; *timed_out receives 1 if the wait reported the timeout, else 0.  No tensor-core
 * work is in flight and the context stays usable.  Allocates and frees 4 bytes of device memory, makes
 * `device` current, synchronous.
 */
int ttc_lqr_selftest_bounded_wait(int32_t device, int32_t poll_limit, int32_t* timed_out);

/*
 * Measured FP32 FMA rate of `device` (no counterpart in the paper; it is the denominator of the roofline
 * fraction reported for the kernels that are bound by plain FP32 arithmetic).  Runs a register-only chain of
 * independent FMAs on every SM, best of five timed launches with CUDA events (about 20 ms in all), once with
 * scalar fma.rn.f32 and once with the packed fma.rn.f32x2 the solver's dense loops use; both results in
 * TFLOP/s (2 flops per FMA).  Synchronous; makes `device` current; allocates and frees 4 KB.
 */
int ttc_lqr_measure_fp32_peak(int32_t device, double* tflops_scalar, double* tflops_packed);

/* Free the handle and its workspace (synchronises the handle's device).  NULL is OK. */
int ttc_lqr_destroy(ttc_lqr_handle* h);

/* Small integer facts about the handle (TTC_QUERY_*); returns INVALID_ARGUMENT on a bad key. */
int ttc_lqr_query(const ttc_lqr_handle* h, int32_t key, int64_t* value);

/* Static, human-readable name of a status code. */
const char* ttc_lqr_status_string(int status);

/* Detail of the last error raised on this thread (empty string if none). */
const char* ttc_lqr_last_error(void);

#ifdef __cplusplus
}
#endif
#endif /* TTC_LQR_H_ */
