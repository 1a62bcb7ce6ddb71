// Internal launch interface between the host logic (gn_context.cu) and the kernels.
#pragma once
#include <cuda_runtime.h>
#include <stdint.h>

namespace gn {

// One dense contraction with a fused epilogue:
//
//   acc[m][n] = sum_k A1(m,k) B1(k,n)  (+ sum_k A2(m,k) B2(k,n) when A2 != nullptr)
//   t = acc + bias[n]                   (bias != nullptr)
//   t = 1 / (1 + exp(-t))               (sigmoid)
//   t = t * zc (1 - zc)                 (dsig != nullptr; zc = dsig[((m / dsig_div) % dsig_rows) * ld_dsig + n])
//   t = alpha * t
//   t = t + beta * cin[m * ld_cin + n]  (cin != nullptr)
//   D[m * ldd + n] = t
//
// A operands: a_kmajor -> A(m,k) = A[m * lda + k], else A(m,k) = A[k * lda + m].
// B operands: b_kmajor -> B(k,n) = B[n * ldb + k], else B(k,n) = B[k * ldb + n].
// Both pairs share layouts but have their own K and leading dimensions.
struct GemmArgs {
  int M = 0, N = 0;
  const float* A1 = nullptr; const float* B1 = nullptr; int K1 = 0; int64_t lda1 = 0, ldb1 = 0;
  const float* A2 = nullptr; const float* B2 = nullptr; int K2 = 0; int64_t lda2 = 0, ldb2 = 0;
  // Error-compensated form of the tensor-core kernel (3 x TF32): when A1lo is set, every operand X is given as
  // X = Xhi + Xlo with both parts exactly representable in TF32 (A1, B1, A2, B2 hold the hi parts; same
  // layouts and leading dimensions for the lo parts), and acc = sum Alo Bhi + Ahi Blo + Ahi Bhi.
  const float* A1lo = nullptr; const float* B1lo = nullptr; const float* A2lo = nullptr; const float* B2lo = nullptr;
  bool a1_split_fresh = false;   // caller's word that A1 is, unchanged, the A1 of the previous contraction
  // Error-compensated form: the result will itself be an operand of a later contraction (emit_parts, set by the
  // caller), and where the hi / lo parts of every stored value go (Dhi, Dlo with leading dimension ld_parts,
  // filled in by the host logic that owns the buffers).
  bool emit_parts = false;
  float* Dhi = nullptr; float* Dlo = nullptr; int64_t ld_parts = 0;
  bool a_kmajor = true, b_kmajor = true;
  bool mn_padded = false;  // every MN-major operand is followed by >= 128 readable bytes
  int two_cta = -1;        // tensor-core kernel: -1 choose, 0 one CTA per tile, 1 CTA pair per 256-row tile
  float* D = nullptr; int64_t ldd = 0;
  const float* bias = nullptr;
  bool sigmoid = false;
  const float* dsig = nullptr; int64_t ld_dsig = 0; int dsig_rows = 1; int dsig_div = 1;
  float alpha = 1.f;
  const float* cin = nullptr; int64_t ld_cin = 0; float beta = 0.f;
};

// FP32 fused-multiply-add GEMM (any shape, any alignment).  Returns launches made.
int launch_gemm_ffma(const GemmArgs& g, cudaStream_t st);

// TF32 tensor-core GEMM (tcgen05 + TMA).  Operands must be 16-byte aligned with leading dimensions
// that are multiples of 4 floats (TMA strides); gemm_tf32_eligible says whether a problem qualifies.
// *err_flag receives a non-zero code if a bounded device-side wait ran out.  Returns launches made,
// or -1 if a tensor map could not be encoded.
// sk_ws / sk_flags: optional workspace of gemm_tf32_workspace_floats() floats and
// gemm_tf32_workspace_flags() ints that lets the two-CTA kernel cut the tiles left over after its whole
// waves along K over the CTA pairs; pass nullptr to keep whole tiles.  The flags must be zero before the
// first launch; every launch that completes leaves them zero again (after a launch that gave up on a
// bounded wait they must be cleared by the caller).
bool gemm_tf32_eligible(const GemmArgs& g);
// Error-compensated form (GemmArgs::A1lo ...): whether it takes a problem (the shape must suit the CTA-pair
// kernel; the hi / lo parts must be 16-byte aligned with leading dimensions that are multiples of 4 and be
// followed by >= 128 readable bytes), and its launch.  Returns launches made, or -1 if it cannot run.
bool gemm_tf32x3_eligible(const GemmArgs& g);
int launch_gemm_tf32x3(const GemmArgs& g, int* err_flag, cudaStream_t st);
int64_t gemm_tf32_workspace_floats();
int gemm_tf32_workspace_flags();
int launch_gemm_tf32(const GemmArgs& g, int* err_flag, float* sk_ws, int* sk_flags, cudaStream_t st);
// Up to six problems, each suited to the CTA-pair kernel (M > 128, N >= 128), as ONE launch whose pairs walk a
// common, host-balanced work list.  Whole tiles only.
//   dep_prob == nullptr: independent problems, longest tiles first; the tiles of one fill the partial last wave
//   of another.
//   dep_prob != nullptr: a chain in the given order; problem i reads, as its FIRST A operand (row panels) or, with
//   dep_all[i] != 0, as an operand whose K runs over the producer's rows, the output of problem dep_prob[i] < i
//   (-1: none).  The consumer's tiles wait (bounded) for the producer's, so the layers of a pass overlap instead
//   of each draining the GPU.  `done`: device scratch of n * done_stride ints (done_stride > M / 256 + 1),
//   cleared by the call.
// Returns launches made, or -1 if the group cannot run this way (run the problems one by one, in order).
constexpr int kGemmGroupMax = 6;
bool gemm_tf32_group_eligible(const GemmArgs* gs, int n);
int launch_gemm_tf32_group(const GemmArgs* gs, int n, const int* dep_prob, const int* dep_all, int* done,
                           int done_stride, int* err_flag, cudaStream_t st);

// The work list of such a launch, computed without a device (see gemm_tf32.cu); for tests of the host logic.
int gemm_tf32_plan_group(int n, const int* M, const int* N, const int* K, int pairs, int keep_order, int* counts,
                         int* waves, int* order_out, int* tiles_out);
double gemm_tf32_group_makespan(int n, const int* M, const int* N, const int* K, int keep_order);

// Streaming FP32 kernels for contractions with one dimension <= 16 (the n_L-wide output layer).
// gemm_thin_kind says which of them (if any) takes a problem; THIN_M needs a scratch buffer of
// gemm_thin_scratch_floats(g) floats.  launch_gemm_thin returns the launches made (0 = not taken).
enum ThinKind { THIN_NONE = 0, THIN_N = 1, THIN_M = 2, THIN_K = 3 };
ThinKind gemm_thin_kind(const GemmArgs& g);
int64_t gemm_thin_scratch_floats(const GemmArgs& g);
int launch_gemm_thin(const GemmArgs& g, float* scratch, cudaStream_t st);

// A one-CTA kernel whose bounded wait (limit_ns) can never be satisfied: writes code 9 to *err_flag.
int launch_timeout_probe(int* err_flag, unsigned long long limit_ns, cudaStream_t st);

// ---- vector / memory-bound kernels -------------------------------------------------------------
// Row gather dst[r][:] = src[idx[r]][:]; rows with idx outside [0, src_rows) are zero-filled and
// *err_flag is set to 1.
int launch_gather_rows(const float* src, int64_t src_rows, int cols, const int32_t* idx, int64_t n_idx,
                       float* dst, int* err_flag, cudaStream_t st);

// out[j] = alpha * sum_r A[r * lda + j] + beta * cin[j]  (cin may be nullptr), j < cols.
// scratch: at least colsum_scratch_floats(rows, cols) floats.
int64_t colsum_scratch_floats(int64_t rows, int cols);
int launch_colsum(const float* A, int64_t rows, int cols, int64_t lda, float alpha, const float* cin,
                  float beta, float* out, float* scratch, cudaStream_t st);

// Squared loss and its derivative for a row batch: delta = 2 (Z - Y) (delta may be nullptr),
// partial[b] = sum over the block's elements of (Z - Y)^2 in double.  Returns blocks via *n_partials.
int loss_num_partials(int64_t count);
int launch_loss_delta(const float* Z, const float* Y, int64_t count, float* delta, double* partial,
                      cudaStream_t st);

// Fixed-order double-precision sum of `count` partials: *out (+)= sum.
int launch_sum_partials(const double* partial, int count, double* out, bool accumulate, cudaStream_t st);

// out[i] = a x[i] + b y[i]; out may be x or y.
int launch_axpby(int64_t n, float a, const float* x, float b, const float* y, float* out, cudaStream_t st);

// Two-term TF32 split of a [rows][cols] matrix with leading dimension ld into hi and lo (leading dimension
// ld_out): hi = x rounded to TF32, lo = (x - hi) rounded to TF32, so x = hi + lo up to 2^-22 |x|.
int launch_split_tf32(const float* src, int64_t rows, int cols, int64_t ld, float* hi, float* lo, int64_t ld_out,
                      cudaStream_t st);

// Stored Jacobian factors (d z^L / d s^m per sample, Section 3.3.1).  D is [rows * nL][n] with row i * nL + u.
// factor_last: D[(i, u)][t] = WL[u * n + t] * z (1 - z), z = Zprev[i * n + t]   (layer L-1 from the linear output layer)
int launch_factor_last(const float* WL, const float* Zprev, int64_t rows, int nL, int n, float* D, cudaStream_t st);
// factor_apply, for every neuron group T_b of the layer (groups contiguous, boundaries floor(b n / groups)) and
// every stream a (U and Q hold `streams` matrices [rows][n], stream_stride floats apart):
//   p_u = sum_{j in T_b} D[(i,u)][j] U_a[i][j];  Q_a[i][j] = 2 sum_u D[(i,u)][j] p_u for j in T_b
// (Eqs. direct-JV-cost, JTv; B = 2I).  n_L <= 32.
int launch_factor_apply(const float* D, const float* U, int64_t rows, int nL, int n, int groups, int streams,
                        int64_t stream_stride, float* Q, cudaStream_t st);
int launch_factor_apply_last(const float* WL, const float* Zprev, const float* U, int64_t rows, int nL, int n, float* Q,
                             cudaStream_t st);

// ---- conjugate gradient ------------------------------------------------------------------------
// The n coordinates are cut into chunks, each inside one segment (one segment for the full system,
// one per layer for the block-diagonal systems).  Partial sums are per chunk, combined per segment
// in a fixed order in double precision.
struct CgChunk { int64_t start; int32_t len; int32_t seg; };
constexpr int kCgChunk = 4096;

struct CgSeg {           // per-segment scalars, device resident
  double rho;            // r^T r
  double pq;             // p^T q
  double gnorm2;         // ||g||^2
  float alpha, beta;
  int active;
  int first, count;      // this segment's chunks are entries [first, first + count) of the (segment-sorted) chunk table
  int pad;
};

// Device-resident state of one solve: where the kernels that end in a dot product take their tickets, what the
// last scalar update left for the host (sum of rho over segments, number of active segments), the number of steps
// in which some segment was still active, and the history of squared residual norms.
struct CgControl {
  unsigned int ticket;   // zero between launches
  int steps;
  int hist_len, hist_cap;
  double* hist;
  double out[2];
};

// r = -g, p = r, d = 0, partial[c] = sum r^2; then rho = gnorm2 = sum, active = rho > 0 && (tol <= 0 || tol < 1) per segment
int launch_cg_init(const float* g, float* d, float* r, float* p, const CgChunk* chunks, int n_chunks,
                   double* partial, CgSeg* seg, int n_seg, double tol, CgControl* ctl, cudaStream_t st);
// partial[c] = sum p q; with seg != nullptr also pq = sum, alpha = active ? rho / pq : 0 per segment
// (seg == nullptr: partials only, ctl unused)
int launch_cg_dot(const float* p, const float* q, const CgChunk* chunks, int n_chunks, double* partial,
                  CgSeg* seg, int n_seg, CgControl* ctl, cudaStream_t st);
// d += alpha p, r -= alpha q, partial[c] = sum r^2 (alpha per segment); then rho_new = sum, beta = rho_new / rho,
// rho = rho_new, active &= !(sqrt(rho) <= tol ||g||) per segment
int launch_cg_update(const float* p, const float* q, float* d, float* r, const CgChunk* chunks,
                     int n_chunks, CgSeg* seg, int n_seg, double tol, double* partial, CgControl* ctl, cudaStream_t st);
// p = r + beta p   (beta per segment)
int launch_cg_direction(const float* r, float* p, const CgChunk* chunks, int n_chunks, const CgSeg* seg,
                        cudaStream_t st);

}  // namespace gn
