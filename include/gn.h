/*
 * gn.h - C ABI of the subsampled Gauss-Newton product library for fully-connected networks
 *        on one NVIDIA B200 (sm_100a).
 *
 * The library evaluates, for the regularised squared-loss network problem of
 * "Distributed Newton Methods for Deep Neural Networks" (arXiv 1802.00130),
 *
 *     f(theta)  = theta^T theta / (2C) + (1/l) sum_i || z^{L,i} - y^i ||^2           (Eq. obj-function)
 *     grad f    = theta / C + (1/l) sum_i (J^i)^T 2 (z^{L,i} - y^i)                  (Eq. whole-gradient)
 *     G^S v     = v / C + (1/|S|) sum_{i in S} (J^i)^T B^i J^i v,   B^i = 2 I        (Eq. sampled-Gauss)
 *     Ghat^S v  = the same with J^i replaced, block by block, by the columns that
 *                 belong to one layer (w^m, b^m)                                      (Eq. approx-jaco)
 *
 * and runs conjugate gradient on (G^S + lambda I) d = -g (Eq. sample-gaussnewton) or on the
 * independent per-layer systems (Eq. block-gaussnewton).
 *
 * Network (Section 2.1, Section 3.3.2): widths n_0-n_1-...-n_L; s^m = (W^m)^T z^{m-1} + b^m;
 * z^m = 1/(1+exp(-s^m)) for m < L and z^L = s^L.
 *
 * LAYOUTS.  All matrices are dense, row-major, 32-bit IEEE floats.
 *   theta, v, out, grad, g, d  [n], n = sum_m (n_{m-1} n_m + n_m): for m = 1..L the columns of W^m
 *                              one after another (entry w^m_{tj} at j*n_{m-1} + t of the layer's
 *                              run), then b^m (Section 2.1).  Biases are part of theta: they are
 *                              regularised and the I/C term of G acts on them too.
 *   X [l][n_0], Y [l][n_L]     one row per training instance; Y rows are the label vectors y^i.
 *   idx [|S|]                  32-bit row numbers in [0, l); repeated rows are allowed and count
 *                              once per occurrence (1/|S| uses the array length).
 *
 * POINTERS.  A parameter named d_* is a DEVICE pointer on the context's GPU, h_* a HOST pointer.
 * Device pointers must be 4-byte aligned; 16-byte alignment enables the vectorised paths.
 *
 * OWNERSHIP.  The caller owns every buffer it passes.  dX and dY are borrowed for the lifetime of
 * the context and never written.  theta and idx are copied when set, so the caller may reuse its
 * buffers as soon as the call returns.  Input and output vectors of one call must not overlap.
 * All workspaces (activations, CG vectors, reduction scratch) belong to the context and are
 * released by gn_destroy.
 *
 * STREAMS.  Every kernel and copy is enqueued on the stream given to gn_create.  Calls that return
 * host values (gn_fun, gn_grad with f_host, gn_cg_solve, every *_host variant) synchronise that
 * stream before returning; the others only enqueue.  A context is not thread-safe.
 *
 * ERRORS.  Every call returns a gn_status and never throws or aborts.  Arguments are checked before
 * anything is launched.  gn_last_error gives a human-readable reason for the most recent failure.
 * There is no CPU fallback: without a usable CUDA device gn_create fails with GN_ECUDA.
 */
#ifndef GN_H_
#define GN_H_

#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef struct gn_ctx gn_ctx; /* opaque */

typedef enum {
  GN_OK = 0,
  GN_EINVAL = 1,  /* bad argument (null pointer, non-positive size, index out of range, ...)   */
  GN_ENOMEM = 2,  /* a device or host allocation failed                                         */
  GN_ECUDA = 3,   /* a CUDA call or kernel failed; gn_last_error has the CUDA message           */
  GN_ESTATE = 4,  /* call sequence: theta / subsample not set, or stored activations are stale  */
  GN_ETIMEOUT = 5 /* a bounded device-side wait ran out (tensor-core pipeline); results invalid */
} gn_status;

typedef enum {
  GN_TF32 = 0,         /* contractions on the tensor cores with TF32 operands, FP32 accumulate   */
  GN_FP32_ACCURATE = 1 /* results at FP32 accuracy: error-compensated tensor-core contractions  */
                       /* (3 x TF32 on hi / lo operand parts) where the shape allows, the FP32  */
                       /* FMA GEMM elsewhere; see gn_set_accurate_method                        */
} gn_precision;

/*
 * gn_create - describe the problem of Eq. (obj-function): network widths, C, and the training set.
 *   out          receives the context (set to NULL on failure).
 *   L            number of weight layers (>= 1); widths has L+1 entries n_0..n_L, all >= 1.
 *   C            regularisation parameter, > 0.
 *   l            number of training rows, >= 1.
 *   dX, dY       device, [l][n_0] and [l][n_L], borrowed.
 *   prec         arithmetic of the contractions.
 *   cuda_stream  a cudaStream_t.  NULL: the context creates a blocking stream of its own, which orders itself with
 *                work on the legacy default stream as CUDA's blocking streams do (a stream that can be captured is
 *                needed for the graph replay of small CG solves; the legacy default stream cannot).
 * Errors: GN_EINVAL for bad arguments, GN_ECUDA if no device / wrong architecture, GN_ENOMEM.
 */
gn_status gn_create(gn_ctx** out, int L, const int32_t* widths, double C, int64_t l,
                    const float* dX, const float* dY, gn_precision prec, void* cuda_stream);

/* gn_destroy - release the context and every workspace; NULL is accepted. */
gn_status gn_destroy(gn_ctx* ctx);

/* gn_num_params - n of Section 2.1, or -1 for a NULL context. */
int64_t gn_num_params(const gn_ctx* ctx);

/* gn_last_error - reason for the last non-OK status of this context ("" if none). */
const char* gn_last_error(const gn_ctx* ctx);

/* gn_workspace_bytes - device memory currently owned by the context. */
int64_t gn_workspace_bytes(const gn_ctx* ctx);

/* gn_kernel_launches - number of kernels this context has launched so far (all entry points; the kernels of a
 * replayed graph count as if launched one by one).  gn_graph_replays - CG steps issued as one graph launch. */
int64_t gn_kernel_launches(const gn_ctx* ctx);
int64_t gn_graph_replays(const gn_ctx* ctx);

/*
 * gn_set_batch_rows - number of rows processed at a time by gn_fun / gn_grad, which walk the
 * training set in row batches so that their workspace stays bounded (the single-GPU form of the
 * mini-batch pipelining of Section 6.1).  rows >= 1; values above l are clamped.  Default 32768.
 */
gn_status gn_set_batch_rows(gn_ctx* ctx, int64_t rows);

/*
 * gn_set_blockdiag_method - how gn_Gv_blockdiag (and block-diagonal CG) forms its product.
 *   1  propagate: the perturbation of each layer block is pushed through the layers above it and pulled
 *      back (R-operator form, L streams stacked along rows); no extra memory.
 *   2  stored factors, the paper's own mechanism: d z^L / d s^m is computed once per (theta, subsample) by
 *      the backward recurrence of Section 3.3 and kept (|S| n_L n_m floats per layer, Eq. Jelement-store);
 *      a block product is then the two re-ordered contractions of Section 4.2 around it.  Needs L >= 2 and
 *      n_L <= 16 (GN_EINVAL otherwise).  Fewer operations than 1 when n_L is small, more memory traffic.
 *   0  choose (default): where 2 applies and its factors take at most 32 GB, the factors are built when a
 *      solver may run 8 or more products (gn_cg_solve's max_iter, gn_newton_iter's cg_max) or on the
 *      8th single product on one (theta, subsample), and every later product uses them; building them costs
 *      about as much as five to six products of form 1 and saves about a third of each later product.
 *      Otherwise 1.
 * Both give the same product up to rounding.
 */
gn_status gn_set_blockdiag_method(gn_ctx* ctx, int method);

/*
 * gn_set_accurate_method - how GN_FP32_ACCURATE contexts compute the dense contractions (the paper does not fix a
 * floating-point width; the acceptance bound of this mode is 1e-5 relative L2 against float64).
 *   0  choose (default): the tensor cores in error-compensated form wherever the shape suits the CTA-pair kernel
 *      (more than 128 rows and at least 128 columns of output), the FP32 FMA GEMM elsewhere;
 *   1  the FP32 FMA GEMM for everything;
 *   2  same as 0.
 * Error-compensated form: every operand X is split into X = Xhi + Xlo, both exactly representable in TF32
 * (|X - Xhi - Xlo| <= 2^-22 |X|); the product is Alo Bhi + Ahi Blo + Ahi Bhi accumulated in FP32, with the sum over k
 * cut into chunks of 128 terms that are added in FP32 round-to-nearest outside the tensor core (its own accumulator
 * truncates).  Splits of theta and of the stored activations are kept until set_theta / set_subsample; they
 * double the memory those take.  If the kernel cannot be launched on this device or a split buffer cannot be
 * allocated, the contraction runs on the FP32 FMA GEMM instead.  No effect on GN_TF32 contexts.  GN_EINVAL for
 * another value.
 */
gn_status gn_set_accurate_method(gn_ctx* ctx, int method);

/*
 * gn_set_split - variable partition of Section 3.1 for the block-diagonal product and its CG.
 *   split  HOST array of L+1 counts: layer m's n_m neurons are cut into split[m] contiguous groups, group g
 *          holding neurons floor(g n_m / split[m]) .. floor((g+1) n_m / split[m]) - 1 (the paper gives only the
 *          counts, e.g. 3-2-3 for 150-200-30, and equal group sizes in its example).  1 <= split[m] <= n_m.
 * A partition is the weights w^m_{tj} with t in one group of layer m-1 and j in one group of layer m; b^m_j
 * belongs to the partition of the FIRST group of layer m-1.  Partitions are numbered layer by layer and inside
 * layer m by a * split[m] + b (a: group below, b: group at layer m); there are sum_m split[m-1] split[m] of
 * them (at most 1024).  gn_Gv_blockdiag then returns Eq. (approx-jaco) with one block per partition and
 * gn_cg_solve(blockdiag = 1) runs one system per partition (Eq. p-linear).  All ones (the default) means one
 * block per layer.  With any split[m] > 1 the product uses the stored Jacobian factors of Sections 3.3.1 and
 * 4.2 (|S| n_L n_m floats per hidden layer, built once per (theta, subsample)); networks with two or more
 * layers then need n_L <= 32.  Group boundaries that are multiples of 4 neurons keep the 16-byte access paths.
 * The vectors keep the layout of theta.  Synchronises the stream.  GN_EINVAL on a bad count.
 */
gn_status gn_set_split(gn_ctx* ctx, const int32_t* split);

/* gn_num_partitions - number of blocks of the block-diagonal system (L until gn_set_split changes it). */
int32_t gn_num_partitions(const gn_ctx* ctx);

/*
 * gn_set_cg_termination - the rule of Section 4.4 for block-diagonal solves: every partition stops as soon as
 * at least cg_min steps have been taken AND at least finished_share of the partitions have met their own stop
 * rule (Eq. cg-stopping-sample); a partition that met it earlier stays frozen meanwhile.  Steps are counted in
 * lock step (all partitions advance together on one GPU).  Defaults cg_min = 0, finished_share = 1 (every
 * partition runs to its own stop rule); the paper's experiments use cg_min = 3.  finished_share in (0, 1].
 */
gn_status gn_set_cg_termination(gn_ctx* ctx, int32_t cg_min, double finished_share);

/*
 * gn_set_theta - copy the model vector (Section 2.1 layout) into the context.  Activations stored
 * by an earlier gn_set_subsample become stale: products return GN_ESTATE until the subsample is
 * set again.
 */
gn_status gn_set_theta(gn_ctx* ctx, const float* d_theta);
gn_status gn_set_theta_host(gn_ctx* ctx, const float* h_theta);

/*
 * gn_set_subsample - choose S (Section 4.3): copies idx, checks every entry on the device
 * (GN_EINVAL and no out-of-range read if one is outside [0, l)), gathers X_S = X[idx, :] and runs
 * the stored forward pass Z_m = sigma(Z_{m-1} W^m + 1 (b^m)^T), m = 1..L (Eq. xtoz), keeping all
 * Z_m for the products.  Needs theta.  nS >= 1.  Synchronises the stream (to report bad indices).
 */
gn_status gn_set_subsample(gn_ctx* ctx, const int32_t* d_idx, int64_t nS);
gn_status gn_set_subsample_host(gn_ctx* ctx, const int32_t* h_idx, int64_t nS);

/*
 * gn_fun - f(theta) over all l rows (Eq. obj-function, Eq. thiswork-loss).  Needs theta.
 * The sum over rows and theta^T theta are accumulated in double precision.
 */
gn_status gn_fun(gn_ctx* ctx, double* f_host);

/*
 * gn_grad - grad f over all l rows (Eq. whole-gradient; back-propagation of Eqs. ztox-g to
 * xtow-g-bias starting from 2 (z^L - y), Section 3.4).  Writes d_grad [n]; if f_host is not NULL
 * also returns f from the same forward pass (and synchronises).
 */
gn_status gn_grad(gn_ctx* ctx, float* d_grad, double* f_host);
gn_status gn_grad_host(gn_ctx* ctx, float* h_grad, double* f_host);

/*
 * gn_Gv - out = G^S v (Eq. sampled-Gauss, no lambda): forward directional-derivative pass for
 * J v (R s^m = R z^{m-1} W^m + z^{m-1} V^m + c^m, R z^m = sigma'(s^m) R s^m), multiply by B = 2I
 * (Section 3.1), backward pass for J^T (.) (Section 4.2), then v/C + (1/|S|)(.).
 * Needs theta and a current subsample.  d_v, d_out: device [n], not overlapping.
 */
gn_status gn_Gv(gn_ctx* ctx, const float* d_v, float* d_out);
gn_status gn_Gv_host(gn_ctx* ctx, const float* h_v, float* h_out);

/*
 * gn_Gv_blockdiag - out = Ghat^S v (Eq. gausshat / approx-jaco) with one block per layer
 * (w^m, b^m): block m of the result is v_m/C + (1/|S|) sum_i (J^i_m)^T 2 J^i_m v_m.
 */
gn_status gn_Gv_blockdiag(gn_ctx* ctx, const float* d_v, float* d_out);
gn_status gn_Gv_blockdiag_host(gn_ctx* ctx, const float* h_v, float* h_out);

/*
 * gn_cg_solve - conjugate gradient for (A + lambda I) d = -g, A = G^S (blockdiag == 0, Eq.
 * sample-gaussnewton) or A = Ghat^S (blockdiag != 0, Eq. block-gaussnewton).  Starts from d = 0,
 * no preconditioner.  With blockdiag the L layer systems are solved side by side, each with its
 * own step lengths and its own stop test; a block that has met its test is frozen.
 *   d_g            device [n], the right-hand side's negative (the gradient).
 *   lambda         >= 0 (the Levenberg-Marquardt term of Eq. full-gaussnewton).
 *   max_iter       >= 1, the cap on CG steps (the paper uses 250).
 *   tol            sigma of Eq. (CG-stopping-cond): stop once ||(A + lambda I) d + g|| <= tol ||g||
 *                  (per block with blockdiag); tol <= 0 runs exactly max_iter steps.
 *   d_d            device [n], receives d.
 *   iters_host     optional, receives the number of steps taken (steps at whose start some system was still
 *                  active: a right-hand side of zero, or a residual that reaches exactly zero, ends the count).
 *   d_iterates     optional device [max_iter][n]: row k receives d after step k+1.
 *   resnorm_host   optional host [max_iter+1]: entry k is the residual norm after k steps
 *                  (over all coordinates).
 * The step lengths, the stop tests, the step count and the residual history are computed and kept on the device.
 * With tol <= 0 (and no termination rule set by gn_set_cg_termination) all max_iter steps are enqueued without
 * waiting and the stream is synchronised once, at the end; such a solve of a small problem (less than 120 GFLOP
 * per step) captures its second step as a CUDA graph and replays it, and keeps the graph for later solves of the same
 * shape.  With tol > 0 or a termination rule the host reads two numbers after every step (one synchronisation per
 * step), because it has to stop issuing steps.
 */
gn_status gn_cg_solve(gn_ctx* ctx, const float* d_g, double lambda, int blockdiag, int max_iter,
                      double tol, float* d_d, int* iters_host, float* d_iterates,
                      double* resnorm_host);
gn_status gn_cg_solve_host(gn_ctx* ctx, const float* h_g, double lambda, int blockdiag,
                           int max_iter, double tol, float* h_d, int* iters_host,
                           double* resnorm_host);

/*
 * gn_newton_iter - one iteration of the subsampled Newton method of Algorithm 3 with everything on this
 * GPU (no partitions, no communication):
 *   1. g = grad f(theta) over all rows, f(theta);
 *   2. CG for d on (Ghat^S + lambda I) d = -g (blockdiag != 0, Eq. block-gaussnewton) or on the full
 *      system (Eq. sample-gaussnewton), stop rule of Eq. (CG-stopping-cond) with sigma, at most cg_max steps;
 *   3. d <- beta1 d + beta2 dbar with dbar the previous direction, (beta1, beta2) from the two-variable
 *      system of Eq. (sol-comp) on the full G^S; (1, 0) if its determinant is <= eps (Eq. determinant);
 *   4. back-tracking line search: largest alpha in {1, 1/2, 1/4, ...} with
 *      f(theta + alpha d) <= f(theta) + eta alpha g^T d (Eq. linesearch-condition), at most max_backtrack halvings;
 *   5. rho = (f(theta + alpha d) - f(theta)) / (alpha g^T d + alpha^2/2 d^T G^S d) and the next lambda by
 *      Eq. (LM-rules) with (drop, boost).
 * d_theta [n] is updated in place to theta + alpha d; d_dir [n] holds dbar on entry (all zeros at the first
 * iteration, as the paper prescribes) and the new direction d on return; d_idx / nS choose S_k (Section 4.3).
 * The paper's constants: sigma = 0.001, cg_max = 250, lambda_1 = 1, (drop, boost) = (2/3, 3/2), eps = 1e-5;
 * it leaves eta in (0, 1) open.  Synchronises the stream; the context's theta is the new theta on return and
 * the subsample must be set again before products are asked for.
 */
typedef struct {
  double lambda;      /* lambda_k */
  double sigma;       /* CG tolerance; <= 0 runs exactly cg_max steps */
  double eta;         /* sufficient-decrease constant */
  double eps;         /* determinant guard */
  double drop, boost; /* Levenberg-Marquardt factors */
  int32_t cg_max;
  int32_t blockdiag;
  int32_t max_backtrack;
  int32_t reserved;
} gn_newton_params;

typedef struct {
  double f_before, f_after, alpha, beta1, beta2, rho, gTd, dGd, lambda_next;
  int32_t cg_iters, backtracks;
} gn_newton_report;

gn_status gn_newton_iter(gn_ctx* ctx, float* d_theta, const int32_t* d_idx, int64_t nS, float* d_dir,
                         const gn_newton_params* params, gn_newton_report* report);

/* ======================================================================================================
 * TEST AND MEASUREMENT HOOKS.  Everything from here to gn_debug_option serves the test suite and the
 * benchmark (failure paths, single kernels, per-launch timing, A/B switches); a solver has no use for them.
 * ====================================================================================================== */

/*
 * gn_debug_timeout_probe - test hook for the failure path of the tensor-core pipeline: launches one
 * CTA that waits, with the pipeline's bounded-wait code and the given limit (0 < limit_ms <= 1000), on a
 * barrier nothing arrives on.  The wait runs out, the kernel records its code and returns, and the call
 * reports GN_ETIMEOUT like any synchronising call would after a timed-out GEMM.  The context stays usable.
 */
gn_status gn_debug_timeout_probe(gn_ctx* ctx, double limit_ms);

/*
 * gn_debug_plan_group - the work list a grouped (or chained, keep_order != 0) launch of the CTA-pair kernel would use
 * for n <= 6 contractions of shapes M[i] x N[i] x K[i] on `pairs` (1..80) CTA pairs; host arithmetic only, no device
 * and no context needed.  Outputs, per problem k in LAUNCH order: order[k] = its index in the caller's list, tiles[k] =
 * its 256-row tiles, waves[k] = how many whole waves of them every pair runs (tiles q, q + pairs, ...), and
 * counts[k * pairs + q] = tiles of it that pair q runs in all (host arrays of n, n, n and n * pairs entries).
 * Returns the number of pairs the launch would use, or -1 for bad arguments.
 */
int32_t gn_debug_plan_group(int32_t n, const int32_t* M, const int32_t* N, const int32_t* K, int32_t pairs,
                            int32_t keep_order, int32_t* counts, int32_t* waves, int32_t* order, int32_t* tiles);

/*
 * gn_debug_check_canaries - every device allocation of the context ends in 256 bytes of slack, the last 128 of
 * which are set to a guard pattern when the allocation is made and are never part of any operand.  This call
 * synchronises, reads the guard bytes of every live allocation back and returns GN_ECUDA (with the size of the
 * damaged workspace in gn_last_error) if any of them has changed, i.e. if some kernel wrote past the end of a
 * workspace; *n_checked (optional) receives the number of allocations looked at.  A stand-in, for writes past
 * the end, for a memory checker where none can be run.
 */
gn_status gn_debug_check_canaries(gn_ctx* ctx, int64_t* n_checked);

/*
 * gn_debug_activations - copy the stored Z_m (m in 1..L, [|S|][n_m]) of the current subsample to a
 * device buffer; a test hook for the stored forward pass (Eq. xtoz).
 */
gn_status gn_debug_activations(gn_ctx* ctx, int m, float* d_out);

/*
 * gn_profile - switch per-launch timing of the contraction kernels on (enable != 0) or off.  While on,
 * every GEMM launch is bracketed by a pair of CUDA events on the context's stream.
 * gn_profile_read - synchronise the stream and return, for the CTA-pair tensor-core kernel that carries the large
 * contractions (index 0), the FP32 FMA GEMM (index 1), the streaming kernels for n_L-wide shapes (index 2), the
 * error-compensated tensor-core kernel of GN_FP32_ACCURATE contexts (index 3) and the one-CTA tensor-core kernel
 * that takes the n_L-wide and small-M shapes in TF32 mode (index 4): summed device time in milliseconds,
 * floating-point operations of the contractions (2 M N K per launch, summed over the problems of a grouped
 * launch; for index 3 the three TF32 products per term count once) and number of launches; then reset the
 * counters.  Each output is an array of FIVE entries and may be NULL.
 */
gn_status gn_profile(gn_ctx* ctx, int enable);
gn_status gn_profile_read(gn_ctx* ctx, double* gemm_ms, double* gemm_flop, int64_t* gemm_launches);

/*
 * gn_debug_gemm - test hook: one contraction D[M][N] = sum_k A(m,k) B(k,n) on the context's stream
 * with the kernel of the given kind (0 = tensor-core TF32, 1 = FP32 FMA GEMM, 2 = streaming kernel for
 * a dimension <= 16, 3 = tensor-core TF32 with the promise that every [K][M] / [K][N] operand is
 * followed by at least 128 readable bytes, which lets it fetch them with one TMA box per stage;
 * 4 and 5 = as 3 with one CTA per 128-row tile, respectively a CTA pair per 256-row tile, forced;
 * 6 = as 5 but whole tiles only, i.e. without the stream-K split of tiles between CTA pairs;
 * 7 = the error-compensated tensor-core form of GN_FP32_ACCURATE contexts, see gn_set_accurate_method).  a_kmajor: A is [M][K]
 * (else [K][M]); b_kmajor: B is [N][K] (else [K][N]); all row-major with the given leading
 * dimensions.  GN_EINVAL if the chosen kernel cannot take the operands (alignment, shape).
 */
gn_status gn_debug_gemm(gn_ctx* ctx, int kind, int M, int N, int K, const float* dA, int64_t lda,
                        int a_kmajor, const float* dB, int64_t ldb, int b_kmajor, float* dD, int64_t ldd);

/*
 * gn_debug_gemm_epilogue - gn_debug_gemm with the epilogue options every contraction kernel of the path takes:
 *   D = alpha * dsig'( f(A B + 1 bias^T) ) + beta * cin,
 * f = logistic sigmoid if `sigmoid` != 0 (Eq. xtoz), else the identity; dsig'(x)_{mn} = x_{mn} z_{mn} (1 - z_{mn}) with
 * z = d_dsig (the sigmoid derivative of Eq. ztox-g from stored activations) if d_dsig != NULL, else x; d_bias is
 * [N], d_dsig and d_cin are [M][ld_*] row-major device arrays, each may be NULL (cin == NULL: no accumulate term).
 * The path itself uses one option at a time (plus the bias); this hook lets a test put every combination through
 * every kernel.  Errors as gn_debug_gemm; GN_EINVAL also for a leading dimension below N.
 */
gn_status gn_debug_gemm_epilogue(gn_ctx* ctx, int kind, int M, int N, int K, const float* dA, int64_t lda, int a_kmajor,
                                 const float* dB, int64_t ldb, int b_kmajor, float* dD, int64_t ldd, const float* d_bias,
                                 int sigmoid, const float* d_dsig, int64_t ld_dsig, float alpha, const float* d_cin,
                                 int64_t ld_cin, float beta);

/*
 * gn_debug_option - test and measurement hook: switch a launch strategy of the context for A/B runs.
 * option 0: independent contractions of a layer issued as one launch of the CTA-pair kernel (value 0 =
 * one launch per contraction); option 1: cutting left-over tiles along K between CTA pairs (value 0 = whole
 * tiles only; cannot be switched back on); option 2: failure injection on the host: the value-th device allocation
 * the context asks for from now on is refused as if the device were out of memory (0 = off); nothing on the
 * device is touched by it; option 3: the bias column sums and the n_L-row weight block of a layer on a side stream
 * next to the layer's large contractions (value 0 = everything on the context's stream); option 4: consecutive
 * layers of a pass as one launch whose tiles wait for the tiles they read (value 0 = one launch per layer, 1 = the
 * stored forward pass, the default, 2 = also the forward R pass of a product).  Option 5 (GN_FP32_ACCURATE contexts): the error-compensated kernel also writes the hi / lo parts
 * of a result that a later contraction takes as an operand (value 0 = a separate pass splits it).  Option 6: fixed-length
 * CG solves of small problems replay one captured step as a CUDA graph (value 0 = plain launches).  Option 7: the
 * weight blocks of the stored-factor block product as two chained parts of the subsample's rows (value 0 = one
 * contraction per block; the two forms differ in the order of two partial sums, i.e. by rounding).  Option 8: the
 * hidden layers of a backward pass (full product, gradient) as one chained launch (value 0 = one grouped launch
 * per layer, 1 = always, 2 = for passes of few rows, where it is the faster form: the default).  Option 9: in the
 * stored-factor block product the factor of the last hidden layer, W^L * sigma'(z^{L-1}), is formed on the fly from
 * W^L and the stored activations instead of being read back (value 0 = read back; same bits either way).  Results do not depend on options 0, 3, 4, 5, 6, 9 and, with whole tiles (option 1 off), 8 (tiles, sums
 * and parts are computed identically); GN_EINVAL for an unknown option.
 */
gn_status gn_debug_option(gn_ctx* ctx, int option, int value);

/* ======================================================================================================
 * CONTEXT-FREE ENTRY POINT
 * ====================================================================================================== */

/*
 * gn_thin_m_gemm_noalloc - D[M][N] = sum_r A[r][m] B[r][n] for M <= 16 (the shape of the output layer's
 * weight block, rows = |S| or a row batch) without a context and without allocating anything.
 * The paper has no counterpart to this call; it exists for callers that must not allocate device memory
 * while they run: code living inside a host application whose own allocator holds all of the GPU's memory
 * (a cudaMalloc from a library would fail or fragment it), jobs started under a fixed device-memory
 * budget, and latency-critical loops that cannot take the device-wide synchronisation an allocation may
 * cause.  It runs the same two kernels as the context's thin-M path (gn_debug_gemm kind 2 with both
 * operands row-major over r); only the scratch differs: the per-row-chunk partial sums go to an 8 MiB
 * array that is part of the library image (every GPU that loads the library holds it until the process
 * exits) instead of a cudaMalloc'ed buffer.
 *   M, N, rows     1 <= M <= 16; N a multiple of 4; rows >= 1.
 *   dA             device [rows][lda], lda >= M: A[r][m].
 *   dB             device [rows][ldb], ldb >= N, a multiple of 4, 16-byte aligned: B[r][n].
 *   dD             device [M][ldd], ldd >= N: the result; must not overlap dA or dB.
 *   cuda_stream    stream to enqueue on (NULL = legacy default stream); the call does not synchronise.
 *   errbuf         optional host buffer of errbuf_len bytes that receives the reason for a failure.
 * Limit: (row chunks) x M x N <= 2 097 152 floats, where row chunks = min(ceil(296 / ceil(N/512)),
 * ceil(rows/64)); a larger problem returns GN_EINVAL and launches nothing (e.g. M = 10, N = 2000 fits for
 * any rows; M = 16, N = 4096 does not once rows > 2048).
 * The first call on each device looks up the array's device address (cudaGetSymbolAddress) with that
 * device current; make that first call outside any stream capture.  No cudaMalloc, cudaFree or other
 * allocating routine is called, on the first call or later.  The array is not the caller's to provide, but it is
 * device memory all the same: the CUDA runtime places the library's kernels and this array on a device when the
 * library is first used there (with CUDA's default lazy loading that can be as late as this first call), and a
 * host application that has already taken every free byte leaves no room for that.  So make one call at start-up,
 * before the host application's allocator takes the device's memory: it doubles as the warm-up, and every later
 * call leaves the device's free memory exactly as it found it.
 * All calls share the one array, which keeps the previous call's partial sums: every element that a call
 * reads it has written first, so nothing needs clearing, but two calls whose kernels may overlap on the
 * GPU (different streams, or different host threads) race on it - serialise them.
 */
gn_status gn_thin_m_gemm_noalloc(int M, int N, int64_t rows, const float* dA, int64_t lda, const float* dB,
                                 int64_t ldb, float* dD, int64_t ldd, void* cuda_stream, char* errbuf,
                                 int64_t errbuf_len);

#ifdef __cplusplus
}
#endif
#endif /* GN_H_ */
