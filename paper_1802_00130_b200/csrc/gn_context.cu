// Host side of the C ABI (include/gn.h): context, workspaces, and the launch sequences for the
// stored forward pass, f / gradient over row batches, the full and block-diagonal Gauss-Newton
// products, and conjugate gradient.
#include <algorithm>
#include <cstdio>
#include <cstring>
#include <new>
#include <string>
#include <vector>

#include "../../include/gn.h"
#include "gn_kernels.h"

// Named ranges around the phases of the path (stored forward pass, f / gradient, products, CG solve) for timeline
// tools; compiled in only with -DGN_NVTX (paper_1802_00130_b200/build.py: GN_NVTX=1 in the environment).
#ifdef GN_NVTX
#include <nvtx3/nvToolsExt.h>
namespace {
struct PhaseRange {
  explicit PhaseRange(const char* name) { nvtxRangePushA(name); }
  ~PhaseRange() { nvtxRangePop(); }
};
}  // namespace
#define GN_PHASE(name) PhaseRange gn_phase_range_(name)
#else
#define GN_PHASE(name) do { } while (0)
#endif

using namespace gn;

struct gn_ctx {
  int L = 0;
  std::vector<int> w;               // n_0..n_L
  double C = 1.0;
  int64_t l = 0;
  const float* dX = nullptr;
  const float* dY = nullptr;
  gn_precision prec = GN_FP32_ACCURATE;
  cudaStream_t st = nullptr;
  // side stream: the bias column sums and the n_L-row weight block of a layer are independent of the layer's large
  // contractions and small enough to run beside them; they are forked off after the layer's delta is ready and
  // joined before the product (or row batch) ends
  cudaStream_t st2 = nullptr;
  cudaEvent_t ev_fork = nullptr, ev_join = nullptr;
  bool side_enabled = true, side_open = false, side_region = false;
  int64_t n = 0;
  std::vector<int64_t> w_off, b_off;  // [m], m = 1..L (entry 0 unused)
  int64_t batch_rows = 32768;
  bool have_theta = false, have_sub = false;

  float* theta = nullptr;
  // subsample
  int64_t nS = 0, capS = 0;
  int32_t* idx = nullptr;
  std::vector<float*> Z;    // Z[0] = X_S, Z[m] = [nS][n_m]
  // RZ[m], DS[m]: forward directional derivatives and backward quantities d(.)/d s^m, [|S|][n_m]; once the
  // propagate form of the block-diagonal product has been asked for they are m |S| rows deep (its L streams
  // stacked along rows), see ensure_stacked
  std::vector<float*> RZ;
  std::vector<float*> DS;
  bool stacked = false;     // RZ / DS hold m * capS rows (else capS rows)
  // stored Jacobian factors d z^L / d s^m on the subsample (block-diagonal product, Section 3.3.1)
  std::vector<float*> DF;   // DF[m] = [nS * n_L][n_m], m = 1..L-1
  int64_t capF = 0;         // rows of S the factor buffers hold
  bool factors_valid = false;
  int bd_method = 0;        // 0 choose, 1 propagate L stacked streams, 2 stored factors
  int bd_expect = 0;        // products the running solver may still ask for (0 outside a solver)
  int bd_count = 0;         // propagate-form products since the factors were last invalidated
  // variable partition (Section 3.1): split[m] contiguous neuron groups in layer m; all ones = one block per layer
  std::vector<int> split;
  bool has_split = false;
  int P = 0;                // number of partitions = sum_m split[m-1] split[m]
  float* SU = nullptr; float* SQ = nullptr; int64_t capSplit = 0;   // per-group right-hand sides and results
  int cg_min = 0;           // termination rule of Section 4.4 for block-diagonal solves
  double cg_share = 1.0;
  // row-batch workspace of f / grad
  int64_t capB = 0;
  std::vector<float*> Zb, Db;
  // reductions
  float* colsum_scratch = nullptr; int64_t colsum_cap = 0;
  float* thin_scratch = nullptr; int64_t thin_cap = 0;
  float* sk_ws = nullptr; int* sk_flags = nullptr;   // stream-K workspace of the tensor-core kernel
  bool sk_enabled = true;
  bool group_enabled = true;   // independent contractions of a layer as one launch (TF32 mode)
  // consecutive layers of a pass as one launch with tile-level dependencies (TF32 mode): 0 never, 1 the stored forward
  // pass (where it measured 8 % faster), 2 also the forward R pass of a product (where cutting left-over tiles along K,
  // which a chained launch does not do, measured as fast or faster)
  int chain_level = 1;
  bool split_k_enabled = true; // weight blocks of the stored-factor product as two chained parts of the rows
  int64_t cut_for_nS = -1, cut_rows = 0;   // rows of the first part, chosen once per subsample size
  bool fly_enabled = true;                 // last hidden layer's factor formed on the fly in the stored-factor product
  int back_chain = 2;                      // hidden layers of a backward pass as one chained launch: 0 never, 1 always, 2 where it pays
  int* chain_ctr = nullptr; int64_t chain_ctr_cap = 0;   // finished-tile counters of such a launch
  // FP32-accurate mode on the tensor cores (3 x TF32): hi / lo parts of the operands
  int acc_method = 0;        // 0 choose (tensor cores where the shape allows), 1 FP32 FMA only, 2 as 0
  bool x3_usable = true;     // cleared if the error-compensated kernel could not be launched
  uint64_t theta_epoch = 1, sub_epoch = 1;   // bumped whenever theta / the stored activations are rewritten
  struct SplitBuf { float* hi = nullptr; float* lo = nullptr; int64_t cap = 0; };
  struct SplitEntry {        // split of a matrix that lives in theta or in the stored Z_m, kept until those change
    const float* src; int64_t rows; int cols; int64_t ld; int kind; uint64_t epoch; SplitBuf buf;
  };
  std::vector<SplitEntry> split_cache;
  struct SplitSlot {         // split of any other operand: one slot per operand role, overwritten by the next use
    const float* src = nullptr; int64_t rows = 0; int cols = 0; int64_t ld = 0; SplitBuf buf;
    uint64_t seq = 0;        // contraction (gemm_seq) that wrote these parts
  };
  SplitSlot split_slot[4];
  // hi / lo parts written by the epilogue of the error-compensated kernel for a result that a later contraction of
  // the SAME launch sequence takes as an operand (R z^m, delta s^m, and their row-batch twins): keyed by the result's
  // address, valid only while parts_epoch stands (every launch sequence that may rewrite those buffers bumps it)
  struct PartsEntry { const float* src = nullptr; int64_t rows = 0; int cols = 0; int64_t ld = 0; uint64_t epoch = 0; SplitBuf buf; };
  std::vector<PartsEntry> parts;
  uint64_t parts_epoch = 1;
  bool parts_enabled = false;  // (measured 7 % slower than a separate splitting pass: off unless asked for)
  uint64_t gemm_seq = 0;     // counts contractions (run_gemm calls)
  double* partial = nullptr; int64_t partial_cap = 0;
  double* dscal = nullptr;   // device: [0] loss, [1] theta^T theta, [2] cg sum rho, [3] cg active
  double* hscal = nullptr;   // pinned mirror
  int* err_flag = nullptr;   // [0] gather index error, [1] tensor-core pipeline timeout code
  int* h_err = nullptr;      // pinned mirror of err_flag
  gn_status sticky = GN_OK;  // a launch-time failure that must surface at the next check
  // CG
  float* cg_r = nullptr; float* cg_p = nullptr; float* cg_q = nullptr;
  CgControl* cg_ctl = nullptr; CgControl* h_ctl = nullptr;   // device-resident solver state and its pinned mirror
  double* cg_hist = nullptr; int cg_hist_cap = 0;            // squared residual norms, one per step
  // One CG step (product + the three vector kernels) as a CUDA graph, for problems small enough that issuing the
  // step's ~20 launches from the host takes as long as running them: captured from the second step of a
  // fixed-length solve and replayed for the rest; kept across solves while nothing it has baked in changes.
  struct CgGraph {
    cudaGraphExec_t exec = nullptr;
    uint64_t alloc_gen = 0; int64_t nS = 0; float coef = 0.f; const float* d = nullptr; int stored = 0, method = 0, n_seg = 0;
    int64_t launches = 0;
  };
  CgGraph cg_graph[2];
  bool graph_enabled = true, graph_ok = true;
  int64_t graph_replays = 0;
  bool own_stream = false;     // no stream was given: the context made one (stream capture cannot use the legacy default stream)
  uint64_t alloc_gen = 1;      // bumped by every device allocation and release of the context
  float* tmp_a = nullptr; float* tmp_b = nullptr;  // staging for *_host calls
  float* nt[4] = {nullptr, nullptr, nullptr, nullptr};  // Newton iteration: g, d, G d / G dbar, trial theta
  CgChunk* chunks[2] = {nullptr, nullptr}; int n_chunks[2] = {0, 0};
  CgSeg* segs[2] = {nullptr, nullptr}; int64_t segs_cap[2] = {0, 0};   // per-segment scalars: full system, block systems

  // optional per-GEMM timing
  struct EvPair { cudaEvent_t a, b; double flop; int kind; };
  std::vector<EvPair> ev;
  size_t ev_used = 0;
  bool profiling = false;

  int64_t bytes = 0;
  int64_t launches = 0;
  std::string err;
  struct Owned { void* p; int64_t bytes; };
  std::vector<Owned> owned;     // every device allocation of the context with its accounted size
  int fail_alloc_in = 0;        // test hook: the fail_alloc_in-th device allocation from now is refused (0 = off)
};

namespace {

gn_status fail(gn_ctx* c, gn_status s, const std::string& msg) {
  if (c) c->err = msg;
  return s;
}

gn_status cuda_fail(gn_ctx* c, cudaError_t e, const char* where) {
  return fail(c, e == cudaErrorMemoryAllocation ? GN_ENOMEM : GN_ECUDA,
              std::string(where) + ": " + cudaGetErrorString(e));
}

#define GN_CUDA(c, call)                                          \
  do {                                                            \
    cudaError_t e__ = (call);                                     \
    if (e__ != cudaSuccess) return cuda_fail((c), e__, #call);    \
  } while (0)

#define GN_TRY(expr)                      \
  do {                                    \
    gn_status s__ = (expr);               \
    if (s__ != GN_OK) return s__;         \
  } while (0)

constexpr int kCanaryByte = 0xA5;

template <class T>
gn_status dev_alloc(gn_ctx* c, T** p, int64_t count) {
  *p = nullptr;
  if (count <= 0) count = 1;
  if (c->fail_alloc_in > 0 && --c->fail_alloc_in == 0)
    return fail(c, GN_ENOMEM, std::string("device allocation of ") + std::to_string(count * (int64_t)sizeof(T)) + " bytes refused (injected)");
  void* q = nullptr;
  // 256 bytes of slack: the tensor-core kernel's 3-D TMA boxes may read up to 124 bytes past the last
  // row of an MN-major operand
  cudaError_t e = cudaMalloc(&q, (size_t)count * sizeof(T) + 256);
  if (e != cudaSuccess) {
    cudaGetLastError();
    return fail(c, GN_ENOMEM, std::string("cudaMalloc of ") + std::to_string(count * (int64_t)sizeof(T)) + " bytes: " + cudaGetErrorString(e));
  }
  // the last 128 bytes of the slack are a canary: nothing of the library may write there (gn_debug_check_canaries)
  if (cudaMemset(static_cast<char*>(q) + (size_t)count * sizeof(T) + 128, kCanaryByte, 128) != cudaSuccess) {
    cudaGetLastError();
    cudaFree(q);
    return fail(c, GN_ECUDA, "cudaMemset of a fresh allocation failed");
  }
  c->bytes += count * (int64_t)sizeof(T);
  ++c->alloc_gen;
  c->owned.push_back({q, count * (int64_t)sizeof(T)});
  *p = static_cast<T*>(q);
  return GN_OK;
}

// Frees a context allocation (null is fine); the accounted size is the one recorded when it was made.
template <class T>
void dev_free(gn_ctx* c, T*& p, int64_t = 0) {
  if (!p) return;
  for (auto& o : c->owned)
    if (o.p == (void*)p) { c->bytes -= o.bytes; o.p = nullptr; o.bytes = 0; break; }
  cudaFree(p);
  p = nullptr;
  ++c->alloc_gen;
  // keep the registry from growing without bound across many regrowths
  if (c->owned.size() > 4096) {
    size_t k = 0;
    for (size_t i = 0; i < c->owned.size(); ++i) if (c->owned[i].p) c->owned[k++] = c->owned[i];
    c->owned.resize(k);
  }
}

gn_status check_launch(gn_ctx* c, const char* where) {
  if (c->sticky != GN_OK) { gn_status s = c->sticky; c->sticky = GN_OK; return s; }
  cudaError_t e = cudaGetLastError();
  if (e != cudaSuccess) return cuda_fail(c, e, where);
  return GN_OK;
}

// Side stream: everything enqueued on the main stream so far happens before what follows on the side stream.
cudaStream_t side_fork(gn_ctx* c) {
  if (!c->side_enabled || !c->st2) return c->st;
  cudaEventRecord(c->ev_fork, c->st);
  cudaStreamWaitEvent(c->st2, c->ev_fork, 0);
  c->side_open = true;
  return c->st2;
}
// ... and everything on the side stream so far happens before what follows on the main stream.
void side_join(gn_ctx* c) {
  if (!c->side_open) return;
  cudaEventRecord(c->ev_join, c->st2);
  cudaStreamWaitEvent(c->st, c->ev_join, 0);
  c->side_open = false;
}
// A launch sequence that uses the side stream: inside it, every kernel that works in the side stream's scratch
// buffers (column sums, the n_L-row weight block) goes to the side stream, so those buffers have one user at a
// time; the join happens on every way out.
struct SideJoin {
  gn_ctx* c;
  explicit SideJoin(gn_ctx* ctx) : c(ctx) { c->side_region = true; }
  ~SideJoin() { side_join(c); c->side_region = false; }
};

// Before a workspace that side-stream kernels may still read is released.
void quiesce(gn_ctx* c) {
  cudaStreamSynchronize(c->st);
  if (c->st2) cudaStreamSynchronize(c->st2);
}

// Synchronise the stream; also fetch the tensor-core pipeline's timeout word.
gn_status sync(gn_ctx* c, const char* where) {
  cudaError_t e = cudaMemcpyAsync(c->h_err + 1, c->err_flag + 1, sizeof(int), cudaMemcpyDeviceToHost, c->st);
  if (e == cudaSuccess) e = cudaStreamSynchronize(c->st);
  if (e != cudaSuccess) return cuda_fail(c, e, where);
  if (c->h_err[1] != 0) {
    const int code = c->h_err[1];
    cudaMemsetAsync(c->err_flag + 1, 0, sizeof(int), c->st);
    // a launch that gave up may have left arrival counts of its K-sliced tiles behind
    if (c->sk_flags) cudaMemsetAsync(c->sk_flags, 0, sizeof(int) * gemm_tf32_workspace_flags(), c->st);
    return fail(c, GN_ETIMEOUT, std::string(where) + ": a bounded wait in the tensor-core pipeline ran out (role " +
                                    std::to_string(code) + "); results are invalid");
  }
  return GN_OK;
}

gn_status ensure_sk_workspace(gn_ctx* c);

void run_gemm_kind(gn_ctx* c, const GemmArgs& g, int kind, cudaStream_t st = nullptr) {
  if (!st) st = c->st;
  gn_ctx::EvPair* e = nullptr;
  if (c->profiling) {
    if (c->ev_used == c->ev.size()) {
      gn_ctx::EvPair p{};
      if (cudaEventCreate(&p.a) == cudaSuccess && cudaEventCreate(&p.b) == cudaSuccess) c->ev.push_back(p);
    }
    if (c->ev_used < c->ev.size()) {
      e = &c->ev[c->ev_used++];
      e->flop = 2.0 * g.M * (double)g.N * ((double)g.K1 + (g.A2 ? (double)g.K2 : 0.0));
      // the one-CTA tensor-core kernel (n_L-wide and small-M shapes, bound by memory) is counted apart from the
      // CTA-pair kernel that carries the large contractions
      e->kind = (kind == 0 && !(g.two_cta >= 0 ? g.two_cta != 0 : (g.M > 128 && g.N >= 128))) ? 4 : kind;
      cudaEventRecord(e->a, st);
    }
  }
  if (kind == 0) {
    ensure_sk_workspace(c);   // first tensor-core launch of this context: stream-K workspace
    const bool sk = c->sk_enabled && g.two_cta != 2;
    GemmArgs g2 = g;
    if (g2.two_cta == 2) g2.two_cta = 1;
    const int r = launch_gemm_tf32(g2, c->err_flag + 1, sk ? c->sk_ws : nullptr, sk ? c->sk_flags : nullptr, st);
    if (r < 0) { c->sticky = GN_ECUDA; c->err = "cuTensorMapEncodeTiled failed"; }
    else c->launches += r;
  } else if (kind == 3) {
    const int r = launch_gemm_tf32x3(g, c->err_flag + 1, st);
    if (r < 0) { c->sticky = GN_ECUDA; c->err = "the error-compensated tensor-core kernel could not be launched"; c->x3_usable = false; }
    else c->launches += r;
  } else if (kind == 2) {
    c->launches += launch_gemm_thin(g, c->thin_scratch, st);
  } else {
    c->launches += launch_gemm_ffma(g, st);
  }
  if (e) cudaEventRecord(e->b, st);
}

gn_status ensure_sk_workspace(gn_ctx* c) {
  if (!c->sk_ws && c->sk_enabled) {
    if (dev_alloc(c, &c->sk_ws, gemm_tf32_workspace_floats()) != GN_OK ||
        dev_alloc(c, &c->sk_flags, (int64_t)gemm_tf32_workspace_flags()) != GN_OK ||
        cudaMemsetAsync(c->sk_flags, 0, sizeof(int) * gemm_tf32_workspace_flags(), c->st) != cudaSuccess) {
      c->sk_ws = nullptr; c->sk_flags = nullptr; c->sk_enabled = false;
    }
  }
  return c->sk_ws ? GN_OK : GN_ENOMEM;
}

inline int64_t round4(int64_t x) { return (x + 3) & ~(int64_t)3; }

bool split_buf_reserve(gn_ctx* c, gn_ctx::SplitBuf& b, int64_t need) {
  if (need <= b.cap) return true;
  cudaStreamSynchronize(c->st);   // an earlier contraction may still be reading the old buffers
  dev_free(c, b.hi, b.cap); dev_free(c, b.lo, b.cap);
  b.cap = 0;
  if (dev_alloc(c, &b.hi, need) != GN_OK) return false;
  if (dev_alloc(c, &b.lo, need) != GN_OK) { dev_free(c, b.hi, need); return false; }
  b.cap = need;
  return true;
}

// The results whose parts the epilogue writes live in the subsample and row-batch workspaces: when those move,
// the parts kept for their old addresses go.
void drop_parts(gn_ctx* c) {
  for (auto& e : c->parts) { dev_free(c, e.buf.hi); dev_free(c, e.buf.lo); }
  c->parts.clear();
}

// hi / lo parts of the stored matrix [rows][cols] (leading dimension ld) that serves as an operand.  Matrices
// inside theta or inside the stored activations Z_m are split once per set_theta / set_subsample; anything
// else goes through the slot of its operand role (0 = A1, 1 = B1, 2 = A2, 3 = B2) and is split again on every
// use unless the caller vouches (reuse) that the contraction just before this one read this very operand,
// unchanged.  The caller's word is checked: the parts are taken over only if that previous contraction is
// the one that wrote the slot (it may have gone to another kernel and left the slot alone).
constexpr int64_t kMaxTransientSplitFloats = 1500LL * 1000 * 1000;   // 6 GB per part

bool split_operand(gn_ctx* c, const float* src, int64_t rows, int cols, int64_t ld, int role, bool reuse,
                   const float** hi, const float** lo, int64_t* ld_out) {
  const int64_t ldo = round4(cols);
  *ld_out = ldo;
  int kind = 0;
  uint64_t epoch = 0;
  if (src >= c->theta && src < c->theta + c->n) { kind = 1; epoch = c->theta_epoch; }
  else {
    for (int m = 0; m <= c->L && kind == 0; ++m)
      if (c->Z[m] && src >= c->Z[m] && src < c->Z[m] + c->capS * c->w[m]) { kind = 2; epoch = c->sub_epoch; }
  }
  if (kind != 0) {
    // one entry per start address: a matrix that comes back with another shape (a subsample of another
    // size in the same buffers) replaces the old parts instead of adding to them
    gn_ctx::SplitEntry* e = nullptr;
    for (auto& x : c->split_cache)
      if (x.src == src && x.kind == kind) { e = &x; break; }
    if (!e) {
      if (c->split_cache.size() >= 4096) return false;
      gn_ctx::SplitEntry x{};
      x.src = src; x.kind = kind; x.epoch = 0;
      c->split_cache.push_back(x);
      e = &c->split_cache.back();
    }
    if (e->epoch != epoch || e->rows != rows || e->cols != cols || e->ld != ld) {
      e->epoch = 0;
      if (!split_buf_reserve(c, e->buf, rows * ldo)) return false;
      c->launches += launch_split_tf32(src, rows, cols, ld, e->buf.hi, e->buf.lo, ldo, c->st);
      e->rows = rows; e->cols = cols; e->ld = ld; e->epoch = epoch;
    }
    *hi = e->buf.hi; *lo = e->buf.lo;
    return true;
  }
  for (auto& e : c->parts)
    if (e.src == src && e.epoch == c->parts_epoch && e.rows == rows && e.cols == cols && e.ld == ld && e.buf.hi) {
      *hi = e.buf.hi; *lo = e.buf.lo;      // written by the epilogue that produced this operand
      return true;
    }
  if (rows * ldo > kMaxTransientSplitFloats) return false;
  gn_ctx::SplitSlot& sl = c->split_slot[role];
  const bool same = reuse && sl.seq != 0 && sl.seq + 1 == c->gemm_seq && sl.src == src && sl.rows == rows &&
                    sl.cols == cols && sl.ld == ld && sl.buf.hi;
  if (!same) {
    sl.src = nullptr; sl.seq = 0;
    if (!split_buf_reserve(c, sl.buf, rows * ldo)) return false;
    c->launches += launch_split_tf32(src, rows, cols, ld, sl.buf.hi, sl.buf.lo, ldo, c->st);
    sl.src = src; sl.rows = rows; sl.cols = cols; sl.ld = ld;
  }
  sl.seq = c->gemm_seq;
  *hi = sl.buf.hi; *lo = sl.buf.lo;
  return true;
}

// FP32-accurate contraction on the tensor cores: every operand as hi + lo TF32 parts, three products per
// operand pair, accumulation in chunks (gemm_tf32.cu).  False if the problem has to go to the FP32 FMA GEMM.
bool run_gemm_x3(gn_ctx* c, const GemmArgs& g) {
  if (!c->x3_usable || !gemm_tf32x3_eligible(g)) return false;
  GemmArgs h = g;
  const float *hi = nullptr, *lo = nullptr;
  int64_t ldo = 0;
  // stored matrices: A is [M][K] (K-major) or [K][M]; B is [N][K] (K-major) or [K][N]
  if (!split_operand(c, g.A1, g.a_kmajor ? g.M : g.K1, g.a_kmajor ? g.K1 : g.M, g.lda1, 0, g.a1_split_fresh, &hi, &lo, &ldo)) return false;
  h.A1 = hi; h.A1lo = lo; h.lda1 = ldo;
  if (!split_operand(c, g.B1, g.b_kmajor ? g.N : g.K1, g.b_kmajor ? g.K1 : g.N, g.ldb1, 1, false, &hi, &lo, &ldo)) return false;
  h.B1 = hi; h.B1lo = lo; h.ldb1 = ldo;
  if (g.A2) {
    if (!split_operand(c, g.A2, g.a_kmajor ? g.M : g.K2, g.a_kmajor ? g.K2 : g.M, g.lda2, 2, false, &hi, &lo, &ldo)) return false;
    h.A2 = hi; h.A2lo = lo; h.lda2 = ldo;
    if (!split_operand(c, g.B2, g.b_kmajor ? g.N : g.K2, g.b_kmajor ? g.K2 : g.N, g.ldb2, 3, false, &hi, &lo, &ldo)) return false;
    h.B2 = hi; h.B2lo = lo; h.ldb2 = ldo;
  }
  h.mn_padded = true;     // the parts live in context allocations, which carry slack after their last row
  gn_ctx::PartsEntry* pe = nullptr;
  if (g.emit_parts && c->parts_enabled && (int64_t)g.M * round4(g.N) <= kMaxTransientSplitFloats) {
    // the result is an operand later in this launch sequence: have the epilogue write its hi / lo parts as well
    for (auto& e : c->parts)
      if (e.src == g.D) { pe = &e; break; }
    if (!pe && c->parts.size() < 1024) { c->parts.emplace_back(); pe = &c->parts.back(); pe->src = g.D; }
    if (pe) {
      pe->epoch = 0;
      if (split_buf_reserve(c, pe->buf, (int64_t)g.M * round4(g.N))) {
        h.Dhi = pe->buf.hi; h.Dlo = pe->buf.lo; h.ld_parts = round4(g.N);
      } else {
        pe = nullptr;
      }
    }
  }
  run_gemm_kind(c, h, 3);
  if (pe && c->x3_usable) { pe->rows = g.M; pe->cols = g.N; pe->ld = g.ldd; pe->epoch = c->parts_epoch; }
  return true;
}

// Kernel choice: streaming kernels for the n_L-wide shapes (both precisions: they are exact FP32),
// the tensor-core kernel in TF32 mode when TMA can address the operands and, in its error-compensated
// form, in FP32-accurate mode when the shape suits the CTA-pair kernel; else the FP32 FMA GEMM.
void run_gemm(gn_ctx* c, const GemmArgs& g, cudaStream_t st = nullptr) {
  ++c->gemm_seq;
  const ThinKind thin = gemm_thin_kind(g);
  // In TF32 mode the n_L-wide forward products go to the tensor-core kernel as one 32- or 64-column
  // tile: TMA streams A about 2.5x faster than the SIMT streaming kernel does (measured) - once there are enough
  // 128-row tiles to occupy the SMs; below 48 tiles (a CTA walks its whole K range alone, 53 us at K = 4000 whatever
  // the row count) the streaming kernel, one warp per four rows, is the faster one (3000 rows: 3-4 % of a product).
  const bool thin_n_on_tensor = thin == THIN_N && c->prec == GN_TF32 && gemm_tf32_eligible(g) && g.M >= 48 * 128;
  if (thin != THIN_NONE && !thin_n_on_tensor) {
    const int64_t need = gemm_thin_scratch_floats(g);
    if (need > c->thin_cap) {
      quiesce(c);
      dev_free(c, c->thin_scratch, c->thin_cap);
      c->thin_cap = 0;
      if (dev_alloc(c, &c->thin_scratch, need) != GN_OK) { c->sticky = GN_ENOMEM; return; }
      c->thin_cap = need;
    }
    // the n_L-row weight block streams its operands once and shares nothing with the layer's other contraction
    if (thin == THIN_M && c->side_region && !st) st = side_fork(c);
    run_gemm_kind(c, g, 2, st);
    return;
  }
  if (c->prec == GN_FP32_ACCURATE && c->acc_method != 1 && run_gemm_x3(c, g)) return;
  run_gemm_kind(c, g, (c->prec == GN_TF32 && gemm_tf32_eligible(g)) ? 0 : 1, st);
}

// Independent contractions issued together (any order is allowed).  In TF32 mode those that suit the CTA-pair
// kernel go out in launches of up to three problems with a common work list (the tiles of one fill the partial
// last wave of another); everything else runs one after the other, in the order given.
void run_gemm_group(gn_ctx* c, const GemmArgs* gs, int n) {
  constexpr int kMax = 3;      // (more than three independent problems per launch gained nothing measurable)
  bool taken[16] = {false};
  if (n >= 2 && n <= 16 && c->prec == GN_TF32 && c->group_enabled) {
    GemmArgs pick[kMax];
    int idx[kMax], np = 0;
    auto flush = [&]() {
      if (np >= 2 && gemm_tf32_group_eligible(pick, np)) {
        c->gemm_seq += (uint64_t)np;
        gn_ctx::EvPair* e = nullptr;
        if (c->profiling) {
          if (c->ev_used == c->ev.size()) {
            gn_ctx::EvPair p{};
            if (cudaEventCreate(&p.a) == cudaSuccess && cudaEventCreate(&p.b) == cudaSuccess) c->ev.push_back(p);
          }
          if (c->ev_used < c->ev.size()) {
            e = &c->ev[c->ev_used++];
            e->flop = 0.0;
            for (int i = 0; i < np; ++i)
              e->flop += 2.0 * pick[i].M * (double)pick[i].N * ((double)pick[i].K1 + (pick[i].A2 ? (double)pick[i].K2 : 0.0));
            e->kind = 0;
            cudaEventRecord(e->a, c->st);
          }
        }
        const int r = launch_gemm_tf32_group(pick, np, nullptr, nullptr, nullptr, 0, c->err_flag + 1, c->st);
        if (r < 0) { c->sticky = GN_ECUDA; c->err = "cuTensorMapEncodeTiled failed"; }
        else c->launches += r;
        if (e) cudaEventRecord(e->b, c->st);
        for (int i = 0; i < np; ++i) taken[idx[i]] = true;
      }
      np = 0;
    };
    for (int i = 0; i < n; ++i) {
      if (gemm_thin_kind(gs[i]) != THIN_NONE || !gemm_tf32_group_eligible(&gs[i], 1)) continue;
      pick[np] = gs[i]; idx[np] = i; ++np;
      if (np == kMax) flush();
    }
    flush();
  }
  for (int i = 0; i < n; ++i)
    if (i >= 16 || !taken[i]) run_gemm(c, gs[i]);
}

// (the new buffer is obtained before the old one is let go: the solver and the dot products use c->partial
// without asking for it again, so a refused allocation must leave the old buffer in place)
// The layers of a pass, each reading what the one before it writes (dep[i] = index of that earlier problem, -1 for
// none; dep_all[i]: it reads all of that output, not just the rows of its own tile).  In TF32 mode a run of
// consecutive problems that suit the CTA-pair kernel goes out as ONE launch in which a tile starts as soon as the
// tiles it reads are stored, so a layer's first tiles run beside the previous layer's last ones; everything else
// runs one after the other, in the order given (which is a valid order by construction).
void run_gemm_chain(gn_ctx* c, const GemmArgs* gs, const int* dep, const int* dep_all, int n, int level = 1) {
  int i = 0;
  while (i < n) {
    int j = i;
    if (c->prec == GN_TF32 && c->chain_level >= level) {
      while (j < n && j - i < kGemmGroupMax && gemm_thin_kind(gs[j]) == THIN_NONE && gemm_tf32_group_eligible(&gs[j], 1)) ++j;
    }
    if (j - i >= 2) {
      const int cnt = j - i;
      int64_t panels = 0;
      for (int k = i; k < j; ++k) panels = std::max<int64_t>(panels, (gs[k].M + 255) / 256);
      const int stride = (int)panels + 1;
      if (!c->chain_ctr || (int64_t)kGemmGroupMax * stride > c->chain_ctr_cap) {
        quiesce(c);
        dev_free(c, c->chain_ctr);
        c->chain_ctr_cap = 0;
        if (dev_alloc(c, &c->chain_ctr, (int64_t)kGemmGroupMax * stride) == GN_OK) c->chain_ctr_cap = (int64_t)kGemmGroupMax * stride;
      }
      int ldep[kGemmGroupMax], lall[kGemmGroupMax];
      // (what an earlier launch wrote is complete by stream order: no dependency inside this launch)
      for (int k = 0; k < cnt; ++k) { ldep[k] = dep[i + k] < i ? -1 : dep[i + k] - i; lall[k] = dep_all[i + k]; }
      if (c->chain_ctr) {
        gn_ctx::EvPair* e = nullptr;
        if (c->profiling) {
          if (c->ev_used == c->ev.size()) {
            gn_ctx::EvPair pnew{};
            if (cudaEventCreate(&pnew.a) == cudaSuccess && cudaEventCreate(&pnew.b) == cudaSuccess) c->ev.push_back(pnew);
          }
          if (c->ev_used < c->ev.size()) {
            e = &c->ev[c->ev_used++];
            e->flop = 0.0;
            for (int k = i; k < j; ++k)
              e->flop += 2.0 * gs[k].M * (double)gs[k].N * ((double)gs[k].K1 + (gs[k].A2 ? (double)gs[k].K2 : 0.0));
            e->kind = 0;
            cudaEventRecord(e->a, c->st);
          }
        }
        const int r = launch_gemm_tf32_group(gs + i, cnt, ldep, lall, c->chain_ctr, stride, c->err_flag + 1, c->st);
        if (e) cudaEventRecord(e->b, c->st);
        if (r >= 0) {
          c->launches += r + 1;             // (the clearing of the counters counts as a launch)
          c->gemm_seq += (uint64_t)cnt;
          i = j;
          continue;
        }
        if (e) --c->ev_used;                // nothing was launched: drop the event pair
      }
    }
    run_gemm(c, gs[i]);
    ++i;
  }
}

gn_status ensure_partials(gn_ctx* c, int64_t count) {
  if (count <= c->partial_cap) return GN_OK;
  double* fresh = nullptr;
  GN_TRY(dev_alloc(c, &fresh, count));
  cudaStreamSynchronize(c->st);
  dev_free(c, c->partial);
  c->partial = fresh;
  c->partial_cap = count;
  return GN_OK;
}

// Scratch of the column sums: two slots of equal size (slot 1 starts at colsum_cap / 2), so that the sums of two
// layers can run at the same time on two streams.
gn_status ensure_colsum(gn_ctx* c, int64_t rows, int cols) {
  const int64_t need = 2 * ((colsum_scratch_floats(rows, cols) + 3) / 4 * 4);
  if (need <= c->colsum_cap) return GN_OK;
  quiesce(c);
  dev_free(c, c->colsum_scratch, c->colsum_cap);
  c->colsum_cap = 0;
  GN_TRY(dev_alloc(c, &c->colsum_scratch, need));
  c->colsum_cap = need;
  return GN_OK;
}

// First neuron of group g when a layer of n neurons is cut into `groups` contiguous groups.
int group_lo(int n, int groups, int g) { return (int)(((long long)g * n) / groups); }

const float* Wm(const gn_ctx* c, const float* vec, int m) { return vec + c->w_off[m]; }
const float* bm(const gn_ctx* c, const float* vec, int m) { return vec + c->b_off[m]; }

// Eq. (xtoz): Zout[m] = sigma(Zout[m-1] W^m + 1 b^mT), m = 1..L, over `rows` rows; Zout[0] = Z0.
void forward_pass(gn_ctx* c, const float* Z0, int64_t rows, std::vector<float*>& Zout, bool emit_parts = false) {
  std::vector<GemmArgs> gs((size_t)c->L);
  std::vector<int> dep((size_t)c->L), dep_all((size_t)c->L, 0);
  for (int m = 1; m <= c->L; ++m) {
    GemmArgs& g = gs[(size_t)m - 1];
    g.M = (int)rows; g.N = c->w[m];
    g.A1 = m == 1 ? Z0 : Zout[m - 1]; g.lda1 = c->w[m - 1];
    g.B1 = Wm(c, c->theta, m); g.ldb1 = c->w[m - 1]; g.K1 = c->w[m - 1];
    g.a_kmajor = true; g.b_kmajor = true;
    g.D = Zout[m]; g.ldd = c->w[m];
    g.bias = bm(c, c->theta, m);
    g.sigmoid = m < c->L;
    g.emit_parts = emit_parts && m < c->L;   // Z_m is an operand of layer m + 1 and of its weight block
    dep[(size_t)m - 1] = m - 2;          // layer m reads the rows layer m - 1 writes
  }
  run_gemm_chain(c, gs.data(), dep.data(), dep_all.data(), c->L);
}

// Parameter-space half of the backward pass for one layer (Eqs. xtow-g, xtow-g-bias, and their
// Jacobian twins of Section 4.2): out_W = alpha ds^T Zprev + beta cin_W, out_b = alpha 1^T ds + beta cin_b.
GemmArgs weight_block_args(const gn_ctx* c, int m, const float* ds, const float* Zprev, int64_t rows, float alpha,
                           const float* cin, float beta, float* out, bool padded = true) {
  GemmArgs g;
  g.mn_padded = padded;   // ds and Zprev are context-owned (padded) unless the caller says otherwise
  g.M = c->w[m]; g.N = c->w[m - 1];
  g.A1 = ds; g.lda1 = c->w[m]; g.a_kmajor = false;
  g.B1 = Zprev; g.ldb1 = c->w[m - 1]; g.b_kmajor = false;
  g.K1 = (int)rows;
  g.alpha = alpha;
  g.cin = cin + c->w_off[m]; g.ld_cin = c->w[m - 1]; g.beta = beta;
  g.D = out + c->w_off[m]; g.ldd = c->w[m - 1];
  return g;
}

// on_main: on the context's stream, in the second scratch slot, instead of the side stream and the first.
gn_status bias_block(gn_ctx* c, int m, const float* ds, int64_t rows, float alpha, const float* cin, float beta,
                     float* out, bool on_main = false) {
  GN_TRY(ensure_colsum(c, rows, c->w[m]));
  c->launches += launch_colsum(ds, rows, c->w[m], c->w[m], alpha, cin + c->b_off[m], beta, out + c->b_off[m],
                               c->colsum_scratch + (on_main ? c->colsum_cap / 2 : 0), on_main ? c->st : side_fork(c));
  return GN_OK;
}

gn_status weight_block(gn_ctx* c, int m, const float* ds, const float* Zprev, int64_t rows, float alpha,
                       const float* cin, float beta, float* out, bool padded = true) {
  // (the bias sums first: forked to the side stream before the contraction is enqueued, they run beside it)
  GN_TRY(bias_block(c, m, ds, rows, alpha, cin, beta, out));
  run_gemm(c, weight_block_args(c, m, ds, Zprev, rows, alpha, cin, beta, out, padded));
  return GN_OK;
}

// Activation-space half (Eq. communi-g / communi-jaco followed by Eq. ztox-g):
// dst = (ds W^mT) * sigma'(z^{m-1}), rows stacked modulo z_rows.
GemmArgs backward_data_args(const gn_ctx* c, int m, const float* ds, int64_t rows, const float* Zprev, int64_t z_rows,
                            float* dst, bool ds_just_used = false) {
  GemmArgs g;
  g.a1_split_fresh = ds_just_used;   // the weight block of the same layer has just read these very rows of ds
  g.M = (int)rows; g.N = c->w[m - 1];
  g.A1 = ds; g.lda1 = c->w[m]; g.a_kmajor = true;
  g.B1 = Wm(c, c->theta, m); g.ldb1 = c->w[m - 1]; g.b_kmajor = false;
  g.K1 = c->w[m];
  g.dsig = Zprev; g.ld_dsig = c->w[m - 1]; g.dsig_rows = (int)z_rows;
  g.D = dst; g.ldd = c->w[m - 1];
  g.mn_padded = true;     // B is the context's own (padded) copy of theta
  g.emit_parts = ds_just_used;   // in the full product and the gradient, delta s^{m-1} feeds the two contractions of layer m - 1
  return g;
}

// Both halves for layer m from the same ds: the weight block over `w_rows` rows starting at ds_w, and (above the
// first layer) the activation gradient over `d_rows` rows starting at ds_d.  The two contractions are independent.
gn_status layer_backward(gn_ctx* c, int m, const float* ds_w, int64_t w_rows, const float* ds_d, int64_t d_rows,
                         const float* Zprev, int64_t z_rows, float alpha, const float* cin, float beta, float* out,
                         float* dst, bool w_padded = true) {
  GemmArgs gs[2];
  int n = 0;
  gs[n++] = weight_block_args(c, m, ds_w, Zprev, w_rows, alpha, cin, beta, out, w_padded);
  if (m > 1) gs[n++] = backward_data_args(c, m, ds_d, d_rows, Zprev, z_rows, dst, ds_w == ds_d && w_rows == d_rows);
  GN_TRY(bias_block(c, m, ds_w, w_rows, alpha, cin, beta, out));
  run_gemm_group(c, gs, n);
  return GN_OK;
}

// Layers m_top .. 1 of a backward pass over `rows` rows, delta s^{m_top} = ds_top being complete: every layer's
// activation gradient (Eqs. communi-g, ztox-g) into DSbuf[m - 1] and its weight and bias blocks (Eqs. xtow-g,
// xtow-g-bias) into `out`.  In TF32 mode the contractions go out as ONE chain, [activation gradient, weight block] per
// layer: an activation-gradient tile waits for the tiles of its row panel one layer up, a weight block for all of
// them, and the pairs' loads are levelled over the whole pass instead of per layer (one ramp, one exposed
// epilogue and one ragged last round instead of one per layer).  The bias sums of the layers below m_top can
// then only start when the chain has ended.  zprev[m - 1] = z^{m-1}; layer 1 takes w1_rows rows (the caller adds
// the rest) of an operand that is padded or not (w1_padded).
gn_status backward_hidden_layers(gn_ctx* c, int m_top, const float* ds_top, const std::vector<const float*>& zprev,
                                 std::vector<float*>& DSbuf, int64_t rows, float alpha, const float* cin, float beta,
                                 float* out, int64_t w1_rows, bool w1_padded) {
  if (m_top < 1) return GN_OK;
  // One launch instead of one per layer saves the ramp, the exposed last epilogue and the ragged last round of
  // every layer, but it has to end with layer 1's weight block, whose tiles are as long as the pass has rows, and
  // the lower layers' bias sums wait for all of it: measured at 784-2000-2000-2000-10, it wins below about 4000
  // rows (full product 0.40 -> 0.37 ms at 1500 rows, 0.56 -> 0.52 at 3000; 784-300-300-10 0.161 -> 0.143) and loses
  // above (0.94 -> 1.00 at 6000, 1.13 -> 1.30 at 8000).
  int widest = 0;
  for (int m = 1; m <= m_top; ++m) widest = std::max(widest, c->w[m]);
  const bool chain = c->back_chain == 1 || (c->back_chain == 2 && (double)rows * widest <= 7.0e6);
  if (!(c->prec == GN_TF32 && chain && m_top >= 2)) {
    const float* ds = ds_top;
    for (int m = m_top; m >= 1; --m) {
      const int64_t wr = m == 1 ? w1_rows : rows;
      if (m == 1) GN_TRY(weight_block(c, 1, ds, zprev[0], wr, alpha, cin, beta, out, w1_padded));
      else GN_TRY(layer_backward(c, m, ds, wr, ds, rows, zprev[(size_t)m - 1], rows, alpha, cin, beta, out, DSbuf[(size_t)m - 1]));
      if (m > 1) ds = DSbuf[(size_t)m - 1];
    }
    return GN_OK;
  }
  std::vector<GemmArgs> gs;
  std::vector<int> dep, dep_all;
  GN_TRY(bias_block(c, m_top, ds_top, m_top == 1 ? w1_rows : rows, alpha, cin, beta, out));   // (its operand is ready now)
  int producer = -1;                        // index of the problem that writes delta s^m
  const float* ds = ds_top;
  for (int m = m_top; m >= 1; --m) {
    int next_producer = -1;
    if (m > 1) {
      gs.push_back(backward_data_args(c, m, ds, rows, zprev[(size_t)m - 1], rows, DSbuf[(size_t)m - 1], true));
      dep.push_back(producer); dep_all.push_back(0);
      next_producer = (int)gs.size() - 1;
    }
    gs.push_back(weight_block_args(c, m, ds, zprev[(size_t)m - 1], m == 1 ? w1_rows : rows, alpha, cin, beta, out,
                                   m == 1 ? w1_padded : true));
    dep.push_back(producer); dep_all.push_back(1);
    producer = next_producer;
    if (m > 1) ds = DSbuf[(size_t)m - 1];
  }
  run_gemm_chain(c, gs.data(), dep.data(), dep_all.data(), (int)gs.size());
  // (nothing is left to hide these sums behind: they alternate between the side stream and this one, each with its
  // own scratch, so that two of them run at a time)
  for (int m = m_top - 1; m >= 1; --m)
    GN_TRY(bias_block(c, m, DSbuf[(size_t)m], m == 1 ? w1_rows : rows, alpha, cin, beta, out, ((m_top - 1 - m) & 1) != 0));
  return GN_OK;
}

// out = coef v + (1/|S|) J^T (2 J v) over the stored subsample (Eq. sampled-Gauss).
gn_status product_full(gn_ctx* c, const float* v, float* out, float coef) {
  GN_PHASE("G v");
  SideJoin side_guard(c);
  ++c->parts_epoch;
  const int L = c->L;
  const int64_t nS = c->nS;
  {
    std::vector<GemmArgs> gs((size_t)L);
    std::vector<int> dep((size_t)L), dep_all((size_t)L, 0);
    for (int m = 1; m <= L; ++m) {
      GemmArgs& g = gs[(size_t)m - 1];
      g.M = (int)nS; g.N = c->w[m];
      if (m == 1) {
        g.A1 = c->Z[0]; g.lda1 = c->w[0]; g.B1 = Wm(c, v, 1); g.ldb1 = c->w[0]; g.K1 = c->w[0];
      } else {
        g.A1 = c->RZ[m - 1]; g.lda1 = c->w[m - 1]; g.B1 = Wm(c, c->theta, m); g.ldb1 = c->w[m - 1]; g.K1 = c->w[m - 1];
        g.A2 = c->Z[m - 1];  g.lda2 = c->w[m - 1]; g.B2 = Wm(c, v, m);        g.ldb2 = c->w[m - 1]; g.K2 = c->w[m - 1];
      }
      g.bias = bm(c, v, m);
      if (m < L) { g.dsig = c->Z[m]; g.ld_dsig = c->w[m]; g.dsig_rows = (int)nS; }
      else g.alpha = 2.f;                                   // B = 2I
      g.D = c->RZ[m]; g.ldd = c->w[m];
      g.emit_parts = m < L;              // R z^m is an operand of layer m + 1
      dep[(size_t)m - 1] = m - 2;        // R z^{m-1} of the layer below
    }
    run_gemm_chain(c, gs.data(), dep.data(), dep_all.data(), L, 2);
  }
  const float inv = (float)(1.0 / (double)nS);
  std::vector<const float*> zprev((size_t)L);
  for (int m = 1; m <= L; ++m) zprev[(size_t)m - 1] = c->Z[m - 1];
  // the output layer (streaming kernels at n_L <= 16) on its own, the hidden layers as one pass
  GN_TRY(layer_backward(c, L, c->RZ[L], nS, c->RZ[L], nS, c->Z[L - 1], nS, inv, v, coef, out, L > 1 ? c->DS[L - 1] : nullptr));
  if (L > 1) GN_TRY(backward_hidden_layers(c, L - 1, c->DS[L - 1], zprev, c->DS, nS, inv, v, coef, out, nS, true));
  return check_launch(c, "G v");
}

// Eq. (approx-jaco), one block per layer.  The perturbation of layer k is pushed to the output and
// pulled back to layer k only; the L streams are stacked along rows, stream j occupying rows
// [(j-1)|S|, j|S|) of every buffer at or above layer j, so each layer runs one stacked GEMM.
// The propagate form stacks its L streams along rows: the first time it is asked for, RZ_m and DS_m are regrown
// to m |S| rows (contexts that only ever use the full product and the stored factors never pay for that).
gn_status ensure_stacked(gn_ctx* c) {
  if (c->stacked) return GN_OK;
  quiesce(c);
  drop_parts(c);
  for (int m = 1; m <= c->L; ++m) { dev_free(c, c->RZ[m]); dev_free(c, c->DS[m]); }
  c->stacked = true;
  for (int m = 1; m <= c->L; ++m) {
    gn_status st = dev_alloc(c, &c->RZ[m], (int64_t)m * c->capS * c->w[m]);
    if (st == GN_OK && m < c->L) st = dev_alloc(c, &c->DS[m], (int64_t)m * c->capS * c->w[m]);
    if (st != GN_OK) {
      // leave a consistent, empty state: the next set_subsample allocates afresh
      for (int k = 1; k <= c->L; ++k) { dev_free(c, c->RZ[k]); dev_free(c, c->DS[k]); }
      for (int k = 0; k <= c->L; ++k) dev_free(c, c->Z[k]);
      dev_free(c, c->idx);
      c->capS = 0; c->have_sub = false; c->factors_valid = false;
      return st;
    }
  }
  return GN_OK;
}

gn_status product_blockdiag(gn_ctx* c, const float* v, float* out, float coef) {
  GN_TRY(ensure_stacked(c));
  SideJoin side_guard(c);
  ++c->parts_epoch;
  const int L = c->L;
  const int64_t nS = c->nS;
  for (int k = 1; k <= L; ++k) {
    // the streams that entered below layer k move up one layer; stream k enters (disjoint rows of R z^k: independent)
    GemmArgs gs[2];
    int n = 0;
    if (k > 1) {
      GemmArgs& g = gs[n++];
      g.M = (int)((k - 1) * nS); g.N = c->w[k];
      g.A1 = c->RZ[k - 1]; g.lda1 = c->w[k - 1]; g.B1 = Wm(c, c->theta, k); g.ldb1 = c->w[k - 1]; g.K1 = c->w[k - 1];
      if (k < L) { g.dsig = c->Z[k]; g.ld_dsig = c->w[k]; g.dsig_rows = (int)nS; }
      else g.alpha = 2.f;
      g.D = c->RZ[k]; g.ldd = c->w[k];
    }
    GemmArgs& g = gs[n++];
    g.M = (int)nS; g.N = c->w[k];
    g.A1 = c->Z[k - 1]; g.lda1 = c->w[k - 1]; g.B1 = Wm(c, v, k); g.ldb1 = c->w[k - 1]; g.K1 = c->w[k - 1];
    g.bias = bm(c, v, k);
    if (k < L) { g.dsig = c->Z[k]; g.ld_dsig = c->w[k]; g.dsig_rows = (int)nS; }
    else g.alpha = 2.f;
    g.D = c->RZ[k] + (k - 1) * nS * c->w[k]; g.ldd = c->w[k];
    run_gemm_group(c, gs, n);
  }
  const float* cur = c->RZ[L];
  const float inv = (float)(1.0 / (double)nS);
  for (int k = L; k >= 1; --k) {
    const float* dsk = cur + (k - 1) * nS * c->w[k];
    GN_TRY(layer_backward(c, k, dsk, nS, cur, (k - 1) * nS, c->Z[k - 1], nS, inv, v, coef, out,
                          k > 1 ? c->DS[k - 1] : nullptr));
    if (k > 1) cur = c->DS[k - 1];
  }
  return check_launch(c, "block-diagonal G v");
}

// ---- block-diagonal product through stored factors (the paper's own mechanism, Sections 3.3.1 and 4.2)
bool stored_factors_applicable(const gn_ctx* c) {
  if (c->L < 2 || c->w[c->L] > 16) return false;
  if ((int64_t)c->w[c->L] * c->nS > 65535LL * 128) return false;
  int64_t bytes = 0;
  for (int m = 1; m < c->L; ++m) bytes += (int64_t)c->nS * c->w[c->L] * c->w[m] * 4;
  return bytes <= 32LL * 1000 * 1000 * 1000;
}

// D^{L-1} from the linear output layer, then D^{m-1} = (D^m W^{mT}) * sigma'(z^{m-1}) on |S| n_L rows
// (Eqs. communi-jaco, ztox-jaco, Jelement-store).  Done once per (theta, S).
gn_status ensure_factors(gn_ctx* c) {
  if (c->factors_valid) return GN_OK;
  GN_PHASE("Jacobian factors");
  ++c->parts_epoch;
  const int L = c->L, nL = c->w[L];
  const int64_t nS = c->nS;
  if (nS > c->capF) {
    GN_TRY(sync(c, "factors"));
    for (int m = 1; m < L; ++m) dev_free(c, c->DF[m], c->capF * nL * c->w[m]);
    c->capF = 0;
    for (int m = 1; m < L; ++m) GN_TRY(dev_alloc(c, &c->DF[m], nS * nL * c->w[m]));
    c->capF = nS;
  }
  c->launches += launch_factor_last(Wm(c, c->theta, L), c->Z[L - 1], nS, nL, c->w[L - 1], c->DF[L - 1], c->st);
  for (int m = L - 1; m >= 2; --m) {
    GemmArgs g;
    g.M = (int)(nS * nL); g.N = c->w[m - 1];
    g.A1 = c->DF[m]; g.lda1 = c->w[m]; g.a_kmajor = true;
    g.B1 = Wm(c, c->theta, m); g.ldb1 = c->w[m - 1]; g.b_kmajor = false;
    g.K1 = c->w[m];
    g.dsig = c->Z[m - 1]; g.ld_dsig = c->w[m - 1]; g.dsig_rows = (int)nS; g.dsig_div = nL;
    g.D = c->DF[m - 1]; g.ldd = c->w[m - 1];
    g.mn_padded = true;
    run_gemm(c, g);
  }
  c->factors_valid = true;
  return check_launch(c, "Jacobian factors");
}

gn_status product_blockdiag_stored(gn_ctx* c, const float* v, float* out, float coef) {
  SideJoin side_guard(c);
  ++c->parts_epoch;
  GN_TRY(ensure_factors(c));
  const int L = c->L, nL = c->w[L];
  const int64_t nS = c->nS;
  const float inv = (float)(1.0 / (double)nS);
  constexpr int kGroup = 3;
  // The layers' chains are independent of one another, so each stage is issued for all layers together.
  // 1. u_i = V^{mT} z^{m-1,i} + c^m for every row (the inner sum of Eq. direct-JV-cost); at m = L, D = I and B = 2I
  for (int m0 = 1; m0 <= L; m0 += kGroup) {
    GemmArgs gs[kGroup];
    int n = 0;
    for (int m = m0; m <= L && m < m0 + kGroup; ++m) {
      GemmArgs& g = gs[n++];
      g.M = (int)nS; g.N = c->w[m];
      g.A1 = c->Z[m - 1]; g.lda1 = c->w[m - 1]; g.B1 = Wm(c, v, m); g.ldb1 = c->w[m - 1]; g.K1 = c->w[m - 1];
      g.bias = bm(c, v, m);
      if (m == L) g.alpha = 2.f;
      g.D = c->RZ[m]; g.ldd = c->w[m];
    }
    run_gemm_group(c, gs, n);
  }
  // 2. q_i = D_i^T 2 D_i u_i per sample (Eqs. direct-JV-cost, JTv)
  // (the factor of the last hidden layer is W^L * sigma'(z^{L-1}): formed on the fly where the kernel allows it,
  // the stored copy being needed only as the operand of the recurrence that builds the factors below it)
  for (int m = 1; m < L; ++m) {
    int done = 0;
    if (m == L - 1 && c->fly_enabled)
      done = launch_factor_apply_last(Wm(c, c->theta, L), c->Z[L - 1], c->RZ[m], nS, nL, c->w[m], c->DS[m], c->st);
    if (!done) done = launch_factor_apply(c->DF[m], c->RZ[m], nS, nL, c->w[m], 1, 1, 0, c->DS[m], c->st);
    c->launches += done;
  }
  // 3. the weight and bias blocks.  The bias sums and the n_L-row weight block go first: they run on the side
  // stream beside the large weight blocks, which is only possible if they are forked before those are enqueued.
  for (int m = 1; m <= L; ++m)
    GN_TRY(bias_block(c, m, m < L ? c->DS[m] : c->RZ[m], nS, inv, v, coef, out));
  // The weight blocks are few long tiles (64 of 375 k-blocks per 2000 x 2000 layer at
  // |S| = 12000: 160 tiles on 74 pairs for three layers leave a third of the last round idle), so with a long enough
  // K each block is cut into two parts of the rows: the first writes alpha Z^T Q + beta v, the second adds
  // its alpha Z^T Q to that (a chained launch: a second-part tile waits for the first-part tiles of its row panel).
  // More and shorter tiles fill the rounds better, and a short second part fills them best (the long tiles go
  // first, the short ones level the loads): the cut is the one of 1/2, 5/8, 3/4 of the rows for which the host's
  // work list comes out shortest.  The order of the two partial sums is fixed.
  const bool halves = c->prec == GN_TF32 && c->chain_level >= 1 && c->split_k_enabled && nS >= 4096 && L - 1 >= 1 && L - 1 <= kGroup;
  if (halves) {
    GemmArgs gs[2 * kGroup];
    int dep[2 * kGroup], dep_all[2 * kGroup];
    int n = 0;
    const int nl = L - 1;                                     // the hidden layers' blocks (the n_L-row block is a streaming kernel)
    if (c->cut_for_nS != nS) {
      double best = -1.0;
      for (int eighths = 4; eighths <= 6; ++eighths) {
        const int64_t r = (nS * eighths / 8 + 31) / 32 * 32;  // first part: a whole number of k-blocks
        int Ms[2 * kGroup], Ns[2 * kGroup], Ks[2 * kGroup];
        for (int part = 0; part < 2; ++part)
          for (int m = 1; m <= nl; ++m) {
            const int k = part * nl + m - 1;
            Ms[k] = c->w[m]; Ns[k] = c->w[m - 1]; Ks[k] = (int)(part == 0 ? r : nS - r);
          }
        const double t = gemm_tf32_group_makespan(2 * nl, Ms, Ns, Ks, 1);
        if (t >= 0.0 && (best < 0.0 || t < best)) { best = t; c->cut_rows = r; }
      }
      if (best < 0.0) c->cut_rows = (nS / 2 + 31) / 32 * 32;
      c->cut_for_nS = nS;
    }
    const int64_t h0 = c->cut_rows;
    for (int part = 0; part < 2; ++part)
      for (int m = 1; m <= nl; ++m) {
        const int64_t r0 = part == 0 ? 0 : h0, rows = part == 0 ? h0 : nS - h0;
        GemmArgs g = weight_block_args(c, m, c->DS[m] + r0 * c->w[m], c->Z[m - 1] + r0 * c->w[m - 1], rows, inv,
                                       part == 0 ? v : out, part == 0 ? coef : 1.f, out);
        dep[n] = part == 0 ? -1 : m - 1;                      // the first-half problem of the same layer
        dep_all[n] = 0;
        gs[n++] = g;
      }
    run_gemm(c, weight_block_args(c, L, c->RZ[L], c->Z[L - 1], nS, inv, v, coef, out));
    run_gemm_chain(c, gs, dep, dep_all, n);
  } else {
    for (int m0 = 1; m0 <= L; m0 += kGroup) {
      GemmArgs gs[kGroup];
      int n = 0;
      for (int m = m0; m <= L && m < m0 + kGroup; ++m)
        gs[n++] = weight_block_args(c, m, m < L ? c->DS[m] : c->RZ[m], c->Z[m - 1], nS, inv, v, coef, out);
      run_gemm_group(c, gs, n);
    }
  }
  return check_launch(c, "block-diagonal G v (stored factors)");
}

// Eq. (approx-jaco) for a split structure, in the order of Section 4.2.  Layer m with s_a groups below and s_b
// groups at it: stream a holds U_a = Z_{m-1}[:, T_a] V^m[T_a, :] (+ c^m for the first group, which owns the
// biases); one pass over the stored factors turns every (stream a, group b) slice into
// Q_a[:, T_b] = D[:, :, T_b]^T 2 D[:, :, T_b] U_a[:, T_b]; then out_W[T_a, :] = Z_{m-1}[:, T_a]^T Q_a / |S|.
// At the output layer D = I, so Q_a = 2 U_a.
gn_status product_split(gn_ctx* c, const float* v, float* out, float coef) {
  ++c->parts_epoch;
  const int L = c->L, nL = c->w[L];
  const int64_t nS = c->nS;
  if (L >= 2) {
    if (nL > 32) return fail(c, GN_EINVAL, "a split structure needs n_L <= 32 (stored Jacobian factors)");
    if ((int64_t)nL * nS > 65535LL * 128) return fail(c, GN_EINVAL, "n_L * |S| exceeds 8 388 480 rows");
    GN_TRY(ensure_factors(c));
  }
  int64_t need = 0;
  for (int m = 1; m <= L; ++m) {
    const int64_t f = (int64_t)c->split[m - 1] * nS * c->w[m];
    if (f > need) need = f;
  }
  if (need > c->capSplit) {
    GN_TRY(sync(c, "split workspace"));
    dev_free(c, c->SU, c->capSplit); dev_free(c, c->SQ, c->capSplit);
    c->capSplit = 0;
    GN_TRY(dev_alloc(c, &c->SU, need));
    GN_TRY(dev_alloc(c, &c->SQ, need));
    c->capSplit = need;
  }
  const float inv = (float)(1.0 / (double)nS);
  std::vector<GemmArgs> batch;
  for (int m = 1; m <= L; ++m) {
    const int sa = c->split[m - 1], sb = c->split[m], np = c->w[m - 1], nm = c->w[m];
    const int64_t stride = nS * nm;
    for (int a = 0; a < sa; ++a) {
      const int t0 = group_lo(np, sa, a), t1 = group_lo(np, sa, a + 1);
      GemmArgs g;
      g.M = (int)nS; g.N = nm;
      g.A1 = c->Z[m - 1] + t0; g.lda1 = np; g.B1 = Wm(c, v, m) + t0; g.ldb1 = np; g.K1 = t1 - t0;
      if (a == 0) g.bias = bm(c, v, m);
      if (m == L) g.alpha = 2.f;                          // B = 2I
      g.D = c->SU + a * stride; g.ldd = nm;
      batch.push_back(g);
    }
    // the groups' contractions are independent of one another: up to sixteen at a time to the group launcher
    for (size_t b0 = 0; b0 < batch.size(); b0 += 16) run_gemm_group(c, batch.data() + b0, (int)std::min<size_t>(16, batch.size() - b0));
    batch.clear();
    const float* Q = c->SU;
    if (m < L) {
      c->launches += launch_factor_apply(c->DF[m], c->SU, nS, nL, nm, sb, sa, stride, c->SQ, c->st);
      Q = c->SQ;
    }
    for (int a = 0; a < sa; ++a) {
      const int t0 = group_lo(np, sa, a), t1 = group_lo(np, sa, a + 1);
      GemmArgs g;
      g.mn_padded = true;                                   // both operands are context-owned
      g.M = nm; g.N = t1 - t0;
      g.A1 = Q + a * stride; g.lda1 = nm; g.a_kmajor = false;
      g.B1 = c->Z[m - 1] + t0; g.ldb1 = np; g.b_kmajor = false;
      g.K1 = (int)nS;
      g.alpha = inv;
      g.cin = v + c->w_off[m] + t0; g.ld_cin = np; g.beta = coef;
      g.D = out + c->w_off[m] + t0; g.ldd = np;
      batch.push_back(g);
    }
    for (size_t b0 = 0; b0 < batch.size(); b0 += 16) run_gemm_group(c, batch.data() + b0, (int)std::min<size_t>(16, batch.size() - b0));
    batch.clear();
    GN_TRY(ensure_colsum(c, nS, nm));
    c->launches += launch_colsum(Q, nS, nm, nm, inv, v + c->b_off[m], coef, out + c->b_off[m], c->colsum_scratch, c->st);
  }
  return check_launch(c, "partition-wise G v");
}

// Choosing between the two forms when the caller has not: building the factors costs about as much as
// five to six propagate-form products and saves about a third of each later one, so they are built when
// a solver announces at least kFactorBreakEven products, or once that many single products have been
// asked for on the same (theta, S), counting the one at hand; after that every product uses them.
constexpr int kFactorBreakEven = 8;

gn_status product_blockdiag_any(gn_ctx* c, const float* v, float* out, float coef) {
  GN_PHASE("block-diagonal G v");
  if (c->has_split) return product_split(c, v, out, coef);
  bool stored = c->bd_method == 2;
  if (c->bd_method == 0 && stored_factors_applicable(c))
    stored = c->factors_valid || c->bd_expect >= kFactorBreakEven || c->bd_count + 1 >= kFactorBreakEven;
  if (stored && c->L >= 2 && c->w[c->L] <= 16) return product_blockdiag_stored(c, v, out, coef);
  ++c->bd_count;
  return product_blockdiag(c, v, out, coef);
}

gn_status ensure_batch(gn_ctx* c) {
  const int64_t rows = c->batch_rows < c->l ? c->batch_rows : c->l;
  if (rows <= c->capB) return GN_OK;
  quiesce(c);
  drop_parts(c);
  for (int m = 1; m <= c->L; ++m) { dev_free(c, c->Zb[m], c->capB * c->w[m]); dev_free(c, c->Db[m], c->capB * c->w[m]); }
  c->capB = 0;
  for (int m = 1; m <= c->L; ++m) {
    GN_TRY(dev_alloc(c, &c->Zb[m], rows * c->w[m]));
    GN_TRY(dev_alloc(c, &c->Db[m], rows * c->w[m]));
  }
  c->capB = rows;
  return GN_OK;
}

// f and (optionally) the gradient over all rows in row batches (Section 6.1 in its one-GPU form).
gn_status fun_grad(gn_ctx* c, float* d_grad, double* f_host) {
  GN_PHASE("f / gradient");
  GN_TRY(ensure_batch(c));
  const int L = c->L;
  const int64_t Rb = c->capB;
  const int64_t nb = (c->l + Rb - 1) / Rb;
  const int64_t per_batch = loss_num_partials(Rb * c->w[L]);
  GN_TRY(ensure_partials(c, per_batch * nb + (c->n + kCgChunk - 1) / kCgChunk + 16));
  const float inv_l = (float)(1.0 / (double)c->l);
  const float inv_C = (float)(1.0 / c->C);
  for (int64_t b = 0; b < nb; ++b) {
    const int64_t r0 = b * Rb;
    const int64_t rows = (c->l - r0 < Rb) ? c->l - r0 : Rb;
    const float* X0 = c->dX + r0 * c->w[0];
    ++c->parts_epoch;           // the batch buffers are rewritten
    forward_pass(c, X0, rows, c->Zb, true);
    c->launches += launch_loss_delta(c->Zb[L], c->dY + r0 * c->w[L], rows * c->w[L], d_grad ? c->Db[L] : nullptr,
                                     c->partial + b * per_batch, c->st);
    {
      // only the last batch can be shorter than Rb: zero the partial slots it does not write
      const int used = loss_num_partials(rows * c->w[L]);
      if (used < per_batch)
        GN_CUDA(c, cudaMemsetAsync(c->partial + b * per_batch + used, 0, (per_batch - used) * sizeof(double), c->st));
    }
    if (d_grad) {
      SideJoin side_guard(c);     // the next batch overwrites what the side stream reads
      const float* cin0 = b == 0 ? c->theta : d_grad;
      const float beta0 = b == 0 ? inv_C : 1.f;
      std::vector<const float*> zprev((size_t)L);
      for (int m = 1; m <= L; ++m) zprev[(size_t)m - 1] = m == 1 ? X0 : c->Zb[m - 1];
      // layer 1 reads the caller's X, which has no slack after its last row: in the last batch all but the final
      // 32 rows use the padded fast path, the rest is added by a second, unpadded contraction
      const bool last = r0 + rows == c->l;
      const bool tail = last && rows > 64;
      const int64_t head = tail ? rows - 32 : rows;
      if (L > 1) {
        GN_TRY(layer_backward(c, L, c->Db[L], rows, c->Db[L], rows, c->Zb[L - 1], rows, inv_l, cin0, beta0, d_grad, c->Db[L - 1]));
        GN_TRY(backward_hidden_layers(c, L - 1, c->Db[L - 1], zprev, c->Db, rows, inv_l, cin0, beta0, d_grad, head, tail || !last));
      } else {
        GN_TRY(weight_block(c, 1, c->Db[1], X0, head, inv_l, cin0, beta0, d_grad, tail || !last));
      }
      if (tail)
        GN_TRY(weight_block(c, 1, c->Db[1] + head * c->w[1], X0 + head * c->w[0], 32, inv_l, d_grad, 1.f, d_grad, false));
    }
  }
  if (f_host) {
    c->launches += launch_sum_partials(c->partial, (int)(per_batch * nb), c->dscal + 0, false, c->st);
    // theta^T theta with the CG dot kernel over the single-segment chunk table
    double* tp = c->partial + per_batch * nb;
    c->launches += launch_cg_dot(c->theta, c->theta, c->chunks[0], c->n_chunks[0], tp, nullptr, 0, nullptr, c->st);
    c->launches += launch_sum_partials(tp, c->n_chunks[0], c->dscal + 1, false, c->st);
    GN_CUDA(c, cudaMemcpyAsync(c->hscal, c->dscal, 2 * sizeof(double), cudaMemcpyDeviceToHost, c->st));
    GN_TRY(check_launch(c, "f / grad"));
    GN_TRY(sync(c, "f / grad"));
    *f_host = c->hscal[1] / (2.0 * c->C) + c->hscal[0] / (double)c->l;
    return GN_OK;
  }
  return check_launch(c, "grad");
}

gn_status ensure_tmp(gn_ctx* c) {
  if (!c->tmp_a) GN_TRY(dev_alloc(c, &c->tmp_a, c->n));
  if (!c->tmp_b) GN_TRY(dev_alloc(c, &c->tmp_b, c->n));
  return GN_OK;
}

gn_status need_product_state(gn_ctx* c) {
  if (!c->have_theta) return fail(c, GN_ESTATE, "theta has not been set");
  if (!c->have_sub) return fail(c, GN_ESTATE, "no current subsample (set it after theta)");
  return GN_OK;
}

void push_range(std::vector<CgChunk>& h, int64_t a, int64_t b, int seg) {
  for (int64_t k = a; k < b; k += kCgChunk) {
    CgChunk ch;
    ch.start = k; ch.len = (int32_t)((b - k < kCgChunk) ? b - k : kCgChunk); ch.seg = seg;
    h.push_back(ch);
  }
}

// Chunk table of the block systems.  One block per layer: the layer's run of theta.  With a split structure:
// partition (group a of layer m-1, group b of layer m) owns, in every row j of group b of the stored
// [n_m][n_{m-1}] matrix, the columns of group a; b^m_j goes with the first group of layer m-1.
// Partitions are numbered layer by layer, inside a layer by a * split[m] + b.
void block_chunks(const gn_ctx* c, std::vector<CgChunk>& h) {
  if (!c->has_split) {
    for (int s = 0; s < c->L; ++s) push_range(h, c->w_off[s + 1], s + 1 < c->L ? c->w_off[s + 2] : c->n, s);
    return;
  }
  int base = 0;
  for (int m = 1; m <= c->L; ++m) {
    const int sa = c->split[m - 1], sb = c->split[m], np = c->w[m - 1], nm = c->w[m];
    for (int b = 0; b < sb; ++b) {
      const int j0 = group_lo(nm, sb, b), j1 = group_lo(nm, sb, b + 1);
      if (sa == 1) {
        push_range(h, c->w_off[m] + (int64_t)j0 * np, c->w_off[m] + (int64_t)j1 * np, base + b);
      } else {
        for (int a = 0; a < sa; ++a) {
          const int t0 = group_lo(np, sa, a), t1 = group_lo(np, sa, a + 1);
          for (int j = j0; j < j1; ++j) push_range(h, c->w_off[m] + (int64_t)j * np + t0, c->w_off[m] + (int64_t)j * np + t1, base + a * sb + b);
        }
      }
      push_range(h, c->b_off[m] + j0, c->b_off[m] + j1, base + b);
    }
    base += sa * sb;
  }
}

// Chunk tables are kept sorted by segment, and every segment records where its chunks start, so that the
// per-segment reductions touch only their own partial sums.
gn_status build_chunks(gn_ctx* c, bool block_only) {
  for (int mode = block_only ? 1 : 0; mode < 2; ++mode) {
    std::vector<CgChunk> h;
    if (mode == 0) push_range(h, 0, c->n, 0);
    else block_chunks(c, h);
    std::stable_sort(h.begin(), h.end(), [](const CgChunk& a, const CgChunk& b) { return a.seg < b.seg; });
    const int n_seg = mode == 0 ? 1 : c->P;
    std::vector<CgSeg> segs((size_t)n_seg);
    for (auto& sg : segs) { std::memset(&sg, 0, sizeof(CgSeg)); }
    for (size_t i = 0; i < h.size(); ++i) {
      CgSeg& sg = segs[(size_t)h[i].seg];
      if (sg.count == 0) sg.first = (int)i;
      ++sg.count;
    }
    // room for the partial sums of the new table, then the new tables, then the swap: a refused allocation
    // leaves the old tables (and the structure they belong to) in use
    GN_TRY(ensure_partials(c, 2 * (int64_t)h.size() + 64));
    CgChunk* d_chunks = nullptr;
    CgSeg* d_segs = nullptr;
    gn_status st = dev_alloc(c, &d_chunks, (int64_t)h.size());
    if (st == GN_OK) st = dev_alloc(c, &d_segs, (int64_t)n_seg);
    if (st == GN_OK && (cudaMemcpy(d_chunks, h.data(), h.size() * sizeof(CgChunk), cudaMemcpyHostToDevice) != cudaSuccess ||
                        cudaMemcpy(d_segs, segs.data(), segs.size() * sizeof(CgSeg), cudaMemcpyHostToDevice) != cudaSuccess)) {
      cudaGetLastError();
      st = fail(c, GN_ECUDA, "copy of the chunk tables failed");
    }
    if (st != GN_OK) { dev_free(c, d_chunks); dev_free(c, d_segs); return st; }
    dev_free(c, c->chunks[mode]);
    dev_free(c, c->segs[mode]);
    c->chunks[mode] = d_chunks; c->n_chunks[mode] = (int)h.size();
    c->segs[mode] = d_segs; c->segs_cap[mode] = n_seg;
  }
  return GN_OK;
}

}  // namespace

extern "C" {

gn_status gn_create(gn_ctx** out, int L, const int32_t* widths, double C, int64_t l, const float* dX,
                    const float* dY, gn_precision prec, void* cuda_stream) {
  if (!out) return GN_EINVAL;
  *out = nullptr;
  if (L < 1 || L > 64 || !widths || !(C > 0.0) || l < 1 || !dX || !dY) return GN_EINVAL;
  if (prec != GN_TF32 && prec != GN_FP32_ACCURATE) return GN_EINVAL;
  for (int m = 0; m <= L; ++m)
    if (widths[m] < 1) return GN_EINVAL;
  if (l > 0x7fffffffLL) return GN_EINVAL;
  int dev = 0;
  if (cudaGetDevice(&dev) != cudaSuccess) { cudaGetLastError(); return GN_ECUDA; }
  cudaDeviceProp prop;
  if (cudaGetDeviceProperties(&prop, dev) != cudaSuccess) { cudaGetLastError(); return GN_ECUDA; }
  if (prop.major != 10) return GN_ECUDA;  // kernels are built for sm_100a only
  gn_ctx* c = new (std::nothrow) gn_ctx();
  if (!c) return GN_ENOMEM;
  c->L = L;
  c->w.assign(widths, widths + L + 1);
  c->C = C; c->l = l; c->dX = dX; c->dY = dY; c->prec = prec;
  c->st = static_cast<cudaStream_t>(cuda_stream);
  if (!c->st) {
    // a blocking stream of the context's own: it orders itself with work on the legacy default stream the way
    // CUDA's blocking streams do, so a caller that works on that stream sees no difference
    if (cudaStreamCreate(&c->st) != cudaSuccess) { cudaGetLastError(); delete c; return GN_ECUDA; }
    c->own_stream = true;
  }
  c->w_off.assign(L + 2, 0); c->b_off.assign(L + 2, 0);
  int64_t off = 0;
  for (int m = 1; m <= L; ++m) {
    c->w_off[m] = off; off += (int64_t)c->w[m - 1] * c->w[m];
    c->b_off[m] = off; off += c->w[m];
  }
  c->n = off;
  c->Z.assign(L + 1, nullptr); c->RZ.assign(L + 1, nullptr); c->DS.assign(L + 1, nullptr);
  c->DF.assign(L + 1, nullptr);
  c->Zb.assign(L + 1, nullptr); c->Db.assign(L + 1, nullptr);
  c->split.assign(L + 1, 1); c->has_split = false; c->P = L;
  gn_status s = GN_OK;
  do {
    if ((s = dev_alloc(c, &c->theta, c->n)) != GN_OK) break;
    if ((s = dev_alloc(c, &c->cg_r, c->n)) != GN_OK) break;
    if ((s = dev_alloc(c, &c->cg_p, c->n)) != GN_OK) break;
    if ((s = dev_alloc(c, &c->cg_q, c->n)) != GN_OK) break;
    if ((s = dev_alloc(c, &c->dscal, 16)) != GN_OK) break;
    if ((s = dev_alloc(c, &c->cg_ctl, 1)) != GN_OK) break;
    if (cudaMemset(c->cg_ctl, 0, sizeof(CgControl)) != cudaSuccess) { s = GN_ECUDA; break; }
    if (cudaMallocHost(&c->h_ctl, sizeof(CgControl)) != cudaSuccess) { s = GN_ENOMEM; break; }
    if ((s = dev_alloc(c, &c->err_flag, 2)) != GN_OK) break;
    if (cudaMemset(c->err_flag, 0, 2 * sizeof(int)) != cudaSuccess) { s = GN_ECUDA; break; }
    if (cudaMallocHost(&c->hscal, 16 * sizeof(double)) != cudaSuccess) { s = GN_ENOMEM; break; }
    if (cudaStreamCreateWithFlags(&c->st2, cudaStreamNonBlocking) != cudaSuccess ||
        cudaEventCreateWithFlags(&c->ev_fork, cudaEventDisableTiming) != cudaSuccess ||
        cudaEventCreateWithFlags(&c->ev_join, cudaEventDisableTiming) != cudaSuccess) { s = GN_ECUDA; break; }
    if (cudaMallocHost(&c->h_err, 2 * sizeof(int)) != cudaSuccess) { s = GN_ENOMEM; break; }
    c->h_err[0] = c->h_err[1] = 0;
    if ((s = build_chunks(c, false)) != GN_OK) break;
  } while (0);
  if (s != GN_OK) { gn_destroy(c); return s; }
  *out = c;
  return GN_OK;
}

gn_status gn_destroy(gn_ctx* c) {
  if (!c) return GN_OK;
  quiesce(c);
  for (auto& g : c->cg_graph) if (g.exec) cudaGraphExecDestroy(g.exec);
  if (c->own_stream) cudaStreamDestroy(c->st);
  if (c->st2) cudaStreamDestroy(c->st2);
  if (c->ev_fork) cudaEventDestroy(c->ev_fork);
  if (c->ev_join) cudaEventDestroy(c->ev_join);
  for (auto& o : c->owned)
    if (o.p) cudaFree(o.p);
  for (auto& p : c->ev) { cudaEventDestroy(p.a); cudaEventDestroy(p.b); }
  if (c->hscal) cudaFreeHost(c->hscal);
  if (c->h_ctl) cudaFreeHost(c->h_ctl);
  if (c->h_err) cudaFreeHost(c->h_err);
  cudaGetLastError();
  delete c;
  return GN_OK;
}

int64_t gn_num_params(const gn_ctx* c) { return c ? c->n : -1; }
const char* gn_last_error(const gn_ctx* c) { return c ? c->err.c_str() : "null context"; }
int64_t gn_workspace_bytes(const gn_ctx* c) { return c ? c->bytes : -1; }
int64_t gn_kernel_launches(const gn_ctx* c) { return c ? c->launches : -1; }
int64_t gn_graph_replays(const gn_ctx* c) { return c ? c->graph_replays : -1; }

gn_status gn_set_batch_rows(gn_ctx* c, int64_t rows) {
  if (!c) return GN_EINVAL;
  if (rows < 1) return fail(c, GN_EINVAL, "batch rows must be >= 1");
  c->batch_rows = rows;
  if ((rows < c->l ? rows : c->l) != c->capB && c->capB > 0) {
    // shrink or grow on next use: drop the old workspace now so memory stays bounded
    quiesce(c);
    drop_parts(c);
    for (int m = 1; m <= c->L; ++m) { dev_free(c, c->Zb[m], c->capB * c->w[m]); dev_free(c, c->Db[m], c->capB * c->w[m]); }
    c->capB = 0;
  }
  return GN_OK;
}

gn_status gn_set_blockdiag_method(gn_ctx* c, int method) {
  if (!c) return GN_EINVAL;
  if (method < 0 || method > 2) return fail(c, GN_EINVAL, "method must be 0 (choose), 1 (propagate) or 2 (stored factors)");
  if (method == 2 && (c->L < 2 || c->w[c->L] > 16))
    return fail(c, GN_EINVAL, "stored factors need at least two layers and n_L <= 16");
  c->bd_method = method;
  return GN_OK;
}

gn_status gn_set_accurate_method(gn_ctx* c, int method) {
  if (!c) return GN_EINVAL;
  if (method < 0 || method > 2) return fail(c, GN_EINVAL, "method must be 0 (choose), 1 (FP32 FMA) or 2 (3 x TF32 where the shape allows)");
  c->acc_method = method;
  return GN_OK;
}

gn_status gn_set_split(gn_ctx* c, const int32_t* split) {
  if (!c) return GN_EINVAL;
  if (!split) return fail(c, GN_EINVAL, "split is NULL");
  int64_t P = 0;
  bool any = false;
  for (int m = 0; m <= c->L; ++m) {
    if (split[m] < 1 || split[m] > c->w[m]) return fail(c, GN_EINVAL, "split[m] must lie in [1, n_m]");
    if (split[m] > 1) any = true;
    if (m >= 1) P += (int64_t)split[m - 1] * split[m];
  }
  if (P > 1024) return fail(c, GN_EINVAL, "more than 1024 partitions");
  if (any && c->L >= 2 && c->w[c->L] > 32) return fail(c, GN_EINVAL, "a split structure needs n_L <= 32 (stored Jacobian factors)");
  GN_TRY(sync(c, "set_split"));
  const std::vector<int> old_split = c->split;
  const bool old_has = c->has_split;
  const int old_P = c->P;
  c->split.assign(split, split + c->L + 1);
  c->has_split = any;
  c->P = (int)P;
  const gn_status st = build_chunks(c, true);
  if (st != GN_OK) { c->split = old_split; c->has_split = old_has; c->P = old_P; }   // the old tables are still in place
  return st;
}

int32_t gn_num_partitions(const gn_ctx* c) { return c ? c->P : -1; }

gn_status gn_set_cg_termination(gn_ctx* c, int32_t cg_min, double finished_share) {
  if (!c) return GN_EINVAL;
  if (cg_min < 0) return fail(c, GN_EINVAL, "cg_min must be >= 0");
  if (!(finished_share > 0.0 && finished_share <= 1.0)) return fail(c, GN_EINVAL, "finished_share must lie in (0, 1]");
  c->cg_min = cg_min; c->cg_share = finished_share;
  return GN_OK;
}

gn_status gn_set_theta(gn_ctx* c, const float* d_theta) {
  if (!c) return GN_EINVAL;
  if (!d_theta) return fail(c, GN_EINVAL, "theta is NULL");
  GN_CUDA(c, cudaMemcpyAsync(c->theta, d_theta, c->n * sizeof(float), cudaMemcpyDeviceToDevice, c->st));
  ++c->theta_epoch;
  c->have_theta = true;
  c->have_sub = false;
  return GN_OK;
}

gn_status gn_set_theta_host(gn_ctx* c, const float* h_theta) {
  if (!c) return GN_EINVAL;
  if (!h_theta) return fail(c, GN_EINVAL, "theta is NULL");
  GN_CUDA(c, cudaMemcpyAsync(c->theta, h_theta, c->n * sizeof(float), cudaMemcpyHostToDevice, c->st));
  ++c->theta_epoch;
  GN_TRY(sync(c, "set_theta_host"));
  c->have_theta = true;
  c->have_sub = false;
  return GN_OK;
}

static gn_status set_subsample_impl(gn_ctx* c, const int32_t* idx, int64_t nS, cudaMemcpyKind kind) {
  GN_PHASE("set_subsample");
  if (!c) return GN_EINVAL;
  if (!idx) return fail(c, GN_EINVAL, "idx is NULL");
  if (nS < 1) return fail(c, GN_EINVAL, "the subsample must have at least one row");
  if (!c->have_theta) return fail(c, GN_ESTATE, "theta has not been set");
  if ((int64_t)c->L * nS > 65535LL * 128) return fail(c, GN_EINVAL, "L * |S| exceeds 8 388 480 rows");
  c->have_sub = false;
  c->factors_valid = false;
  c->bd_count = 0;
  ++c->sub_epoch;             // the stored activations are about to be rewritten
  ++c->parts_epoch;
  if (nS > c->capS) {
    GN_TRY(sync(c, "set_subsample"));
    // the stored activations move: the hi / lo parts kept for matrices inside the old buffers go with them
    for (size_t i = 0; i < c->split_cache.size();) {
      if (c->split_cache[i].kind == 2) {
        dev_free(c, c->split_cache[i].buf.hi, c->split_cache[i].buf.cap);
        dev_free(c, c->split_cache[i].buf.lo, c->split_cache[i].buf.cap);
        c->split_cache.erase(c->split_cache.begin() + (long)i);
      } else {
        ++i;
      }
    }
    drop_parts(c);
    dev_free(c, c->idx, c->capS);
    for (int m = 0; m <= c->L; ++m) dev_free(c, c->Z[m], c->capS * c->w[m]);
    for (int m = 1; m <= c->L; ++m) { dev_free(c, c->RZ[m], m * c->capS * c->w[m]); dev_free(c, c->DS[m], m * c->capS * c->w[m]); }
    c->capS = 0;
    GN_TRY(dev_alloc(c, &c->idx, nS));
    for (int m = 0; m <= c->L; ++m) GN_TRY(dev_alloc(c, &c->Z[m], nS * c->w[m]));
    for (int m = 1; m <= c->L; ++m) {
      const int64_t depth = c->stacked ? m : 1;
      GN_TRY(dev_alloc(c, &c->RZ[m], depth * nS * c->w[m]));
      if (m < c->L) GN_TRY(dev_alloc(c, &c->DS[m], depth * nS * c->w[m]));
    }
    c->capS = nS;
  }
  c->nS = nS;
  GN_CUDA(c, cudaMemcpyAsync(c->idx, idx, nS * sizeof(int32_t), kind, c->st));
  GN_CUDA(c, cudaMemsetAsync(c->err_flag, 0, sizeof(int), c->st));
  c->launches += launch_gather_rows(c->dX, c->l, c->w[0], c->idx, nS, c->Z[0], c->err_flag, c->st);
  GN_CUDA(c, cudaMemcpyAsync(c->h_err, c->err_flag, sizeof(int), cudaMemcpyDeviceToHost, c->st));
  forward_pass(c, c->Z[0], nS, c->Z);
  GN_TRY(check_launch(c, "set_subsample"));
  GN_TRY(sync(c, "set_subsample"));
  if (*c->h_err) return fail(c, GN_EINVAL, "a subsample index lies outside [0, l)");
  c->have_sub = true;
  return GN_OK;
}

gn_status gn_set_subsample(gn_ctx* c, const int32_t* d_idx, int64_t nS) {
  return set_subsample_impl(c, d_idx, nS, cudaMemcpyDeviceToDevice);
}
gn_status gn_set_subsample_host(gn_ctx* c, const int32_t* h_idx, int64_t nS) {
  return set_subsample_impl(c, h_idx, nS, cudaMemcpyHostToDevice);
}

gn_status gn_fun(gn_ctx* c, double* f_host) {
  if (!c) return GN_EINVAL;
  if (!f_host) return fail(c, GN_EINVAL, "f_host is NULL");
  if (!c->have_theta) return fail(c, GN_ESTATE, "theta has not been set");
  return fun_grad(c, nullptr, f_host);
}

gn_status gn_grad(gn_ctx* c, float* d_grad, double* f_host) {
  if (!c) return GN_EINVAL;
  if (!d_grad) return fail(c, GN_EINVAL, "grad is NULL");
  if (!c->have_theta) return fail(c, GN_ESTATE, "theta has not been set");
  return fun_grad(c, d_grad, f_host);
}

gn_status gn_grad_host(gn_ctx* c, float* h_grad, double* f_host) {
  if (!c) return GN_EINVAL;
  if (!h_grad) return fail(c, GN_EINVAL, "grad is NULL");
  if (!c->have_theta) return fail(c, GN_ESTATE, "theta has not been set");
  GN_TRY(ensure_tmp(c));
  GN_TRY(fun_grad(c, c->tmp_b, f_host));
  GN_CUDA(c, cudaMemcpyAsync(h_grad, c->tmp_b, c->n * sizeof(float), cudaMemcpyDeviceToHost, c->st));
  return sync(c, "grad_host");
}

gn_status gn_Gv(gn_ctx* c, const float* d_v, float* d_out) {
  if (!c) return GN_EINVAL;
  if (!d_v || !d_out) return fail(c, GN_EINVAL, "v / out is NULL");
  if (d_v == d_out) return fail(c, GN_EINVAL, "v and out must not overlap");
  GN_TRY(need_product_state(c));
  return product_full(c, d_v, d_out, (float)(1.0 / c->C));
}

gn_status gn_Gv_blockdiag(gn_ctx* c, const float* d_v, float* d_out) {
  if (!c) return GN_EINVAL;
  if (!d_v || !d_out) return fail(c, GN_EINVAL, "v / out is NULL");
  if (d_v == d_out) return fail(c, GN_EINVAL, "v and out must not overlap");
  GN_TRY(need_product_state(c));
  return product_blockdiag_any(c, d_v, d_out, (float)(1.0 / c->C));
}

static gn_status product_host(gn_ctx* c, const float* h_v, float* h_out, bool blockdiag) {
  if (!c) return GN_EINVAL;
  if (!h_v || !h_out) return fail(c, GN_EINVAL, "v / out is NULL");
  GN_TRY(need_product_state(c));
  GN_TRY(ensure_tmp(c));
  GN_CUDA(c, cudaMemcpyAsync(c->tmp_a, h_v, c->n * sizeof(float), cudaMemcpyHostToDevice, c->st));
  const float coef = (float)(1.0 / c->C);
  GN_TRY(blockdiag ? product_blockdiag_any(c, c->tmp_a, c->tmp_b, coef) : product_full(c, c->tmp_a, c->tmp_b, coef));
  GN_CUDA(c, cudaMemcpyAsync(h_out, c->tmp_b, c->n * sizeof(float), cudaMemcpyDeviceToHost, c->st));
  return sync(c, "product_host");
}

gn_status gn_Gv_host(gn_ctx* c, const float* h_v, float* h_out) { return product_host(c, h_v, h_out, false); }
gn_status gn_Gv_blockdiag_host(gn_ctx* c, const float* h_v, float* h_out) { return product_host(c, h_v, h_out, true); }

gn_status gn_cg_solve(gn_ctx* c, const float* d_g, double lambda, int blockdiag, int max_iter, double tol,
                      float* d_d, int* iters_host, float* d_iterates, double* resnorm_host) {
  GN_PHASE("CG solve");
  if (!c) return GN_EINVAL;
  if (!d_g || !d_d) return fail(c, GN_EINVAL, "g / d is NULL");
  if (max_iter < 1) return fail(c, GN_EINVAL, "max_iter must be >= 1");
  if (!(lambda >= 0.0)) return fail(c, GN_EINVAL, "lambda must be >= 0");
  GN_TRY(need_product_state(c));
  const int mode = blockdiag ? 1 : 0;
  const int n_seg = blockdiag ? c->P : 1;
  const CgChunk* ch = c->chunks[mode];
  const int nc = c->n_chunks[mode];
  const float coef = (float)(1.0 / c->C + lambda);
  CgSeg* seg = c->segs[mode];
  // device-resident solver state: ticket, step count, residual history
  if (max_iter + 1 > c->cg_hist_cap) {
    GN_TRY(sync(c, "cg history"));
    dev_free(c, c->cg_hist, c->cg_hist_cap);
    c->cg_hist_cap = 0;
    GN_TRY(dev_alloc(c, &c->cg_hist, (int64_t)max_iter + 1));
    c->cg_hist_cap = max_iter + 1;
  }
  CgControl h0{};
  h0.hist = c->cg_hist; h0.hist_cap = max_iter + 1;
  *c->h_ctl = h0;
  GN_CUDA(c, cudaMemcpyAsync(c->cg_ctl, c->h_ctl, sizeof(CgControl), cudaMemcpyHostToDevice, c->st));
  // The host has to look at the scalars after every step only if something may end the solve early: a stop
  // tolerance, or the termination rule of Section 4.4.  Otherwise all max_iter steps are enqueued without waiting
  // (a system that converges exactly freezes, and the steps after that change nothing).
  const bool rule44 = blockdiag && (c->cg_min > 0 || c->cg_share < 1.0);
  const bool watch = tol > 0.0 || rule44;

  c->launches += launch_cg_init(d_g, d_d, c->cg_r, c->cg_p, ch, nc, c->partial, seg, n_seg, tol, c->cg_ctl, c->st);
  GN_TRY(check_launch(c, "cg init"));
  double active = 1.0;
  if (watch) {
    GN_CUDA(c, cudaMemcpyAsync(c->h_ctl, c->cg_ctl, sizeof(CgControl), cudaMemcpyDeviceToHost, c->st));
    GN_TRY(sync(c, "cg init"));
    active = c->h_ctl->out[1];
  }
  int it = 0;
  c->bd_expect = blockdiag ? max_iter : 0;
  struct Reset { int* p; ~Reset() { *p = 0; } } reset_expect{&c->bd_expect};
  auto one_step = [&]() -> gn_status {
    GN_TRY(blockdiag ? product_blockdiag_any(c, c->cg_p, c->cg_q, coef) : product_full(c, c->cg_p, c->cg_q, coef));
    c->launches += launch_cg_dot(c->cg_p, c->cg_q, ch, nc, c->partial, seg, n_seg, c->cg_ctl, c->st);
    c->launches += launch_cg_update(c->cg_p, c->cg_q, d_d, c->cg_r, ch, nc, seg, n_seg, tol, c->partial, c->cg_ctl, c->st);
    c->launches += launch_cg_direction(c->cg_r, c->cg_p, ch, nc, seg, c->st);
    return check_launch(c, "cg step");
  };
  // Fixed-length solve of a small problem: the step's launches are issued once, into a graph, and replayed.
  double step_flop = 0.0;
  for (int m = 1; m <= c->L; ++m) step_flop += (m == 1 ? 4.0 : 8.0) * (double)c->w[m - 1] * c->w[m] * (double)c->nS;
  const bool use_graph = !watch && !d_iterates && !c->profiling && c->graph_enabled && c->graph_ok && max_iter >= 4 &&
                         step_flop < 120e9;
  gn_ctx::CgGraph& cgg = c->cg_graph[mode];
  while (it < max_iter && active > 0.5) {
    // Section 4.4: all partitions stop once cg_min steps are done and the stated share of them have finished
    if (rule44 && it >= c->cg_min && (double)n_seg - active >= c->cg_share * (double)n_seg) break;
    if (use_graph && it >= 1) {
      // (the first step ran as plain launches: every workspace it needs exists and the stored factors are built)
      const bool fits = cgg.exec && cgg.alloc_gen == c->alloc_gen && cgg.nS == c->nS && cgg.coef == coef && cgg.d == d_d &&
                        cgg.stored == (c->factors_valid ? 1 : 0) && cgg.method == c->bd_method && cgg.n_seg == n_seg;
      if (!fits) {
        if (cgg.exec) { cudaGraphExecDestroy(cgg.exec); cgg.exec = nullptr; }
        const int64_t before = c->launches;
        const uint64_t gen = c->alloc_gen;
        cudaGraph_t graph = nullptr;
        gn_status st = GN_OK;
        if (cudaStreamBeginCapture(c->st, cudaStreamCaptureModeThreadLocal) == cudaSuccess) {
          st = one_step();
          const cudaError_t e = cudaStreamEndCapture(c->st, &graph);
          if (st == GN_OK && e == cudaSuccess && graph && gen == c->alloc_gen &&
              cudaGraphInstantiate(&cgg.exec, graph, 0) == cudaSuccess) {
            cgg.alloc_gen = gen; cgg.nS = c->nS; cgg.coef = coef; cgg.d = d_d; cgg.stored = c->factors_valid ? 1 : 0;
            cgg.method = c->bd_method; cgg.n_seg = n_seg; cgg.launches = c->launches - before;
          } else {
            cgg.exec = nullptr;
          }
          if (graph) cudaGraphDestroy(graph);
          c->launches = before;              // nothing has run yet: the captured step runs when the graph is launched
        }
        cudaGetLastError();
        if (!cgg.exec) {                     // capture is not available here: plain launches from now on
          c->graph_ok = false;
          c->sticky = GN_OK;
          GN_TRY(one_step());
          ++it;
          continue;
        }
      }
      if (c->graph_ok && cgg.exec) {
        GN_CUDA(c, cudaGraphLaunch(cgg.exec, c->st));
        c->launches += cgg.launches;
        ++c->graph_replays;
        ++it;
        continue;
      }
    }
    GN_TRY(one_step());
    if (d_iterates)
      GN_CUDA(c, cudaMemcpyAsync(d_iterates + (int64_t)it * c->n, d_d, c->n * sizeof(float), cudaMemcpyDeviceToDevice, c->st));
    if (watch) {
      GN_CUDA(c, cudaMemcpyAsync(c->h_ctl, c->cg_ctl, sizeof(CgControl), cudaMemcpyDeviceToHost, c->st));
      GN_TRY(sync(c, "cg step"));
      active = c->h_ctl->out[1];
    }
    ++it;
  }
  // one read of the state at the end: steps in which a segment was still active, and the residual history
  GN_CUDA(c, cudaMemcpyAsync(c->h_ctl, c->cg_ctl, sizeof(CgControl), cudaMemcpyDeviceToHost, c->st));
  GN_TRY(sync(c, "cg solve"));
  const int steps = watch ? it : c->h_ctl->steps;
  if (iters_host) *iters_host = steps;
  if (resnorm_host) {
    const int len = c->h_ctl->hist_len < steps + 1 ? c->h_ctl->hist_len : steps + 1;
    GN_CUDA(c, cudaMemcpy(resnorm_host, c->cg_hist, (size_t)len * sizeof(double), cudaMemcpyDeviceToHost));
    for (int k = 0; k < len; ++k) resnorm_host[k] = sqrt(resnorm_host[k]);
  }
  return GN_OK;
}

gn_status gn_cg_solve_host(gn_ctx* c, const float* h_g, double lambda, int blockdiag, int max_iter, double tol,
                           float* h_d, int* iters_host, double* resnorm_host) {
  if (!c) return GN_EINVAL;
  if (!h_g || !h_d) return fail(c, GN_EINVAL, "g / d is NULL");
  GN_TRY(need_product_state(c));
  GN_TRY(ensure_tmp(c));
  GN_CUDA(c, cudaMemcpyAsync(c->tmp_a, h_g, c->n * sizeof(float), cudaMemcpyHostToDevice, c->st));
  GN_TRY(gn_cg_solve(c, c->tmp_a, lambda, blockdiag, max_iter, tol, c->tmp_b, iters_host, nullptr, resnorm_host));
  GN_CUDA(c, cudaMemcpyAsync(h_d, c->tmp_b, c->n * sizeof(float), cudaMemcpyDeviceToHost, c->st));
  return sync(c, "cg_solve_host");
}

gn_status gn_profile(gn_ctx* c, int enable) {
  if (!c) return GN_EINVAL;
  c->profiling = enable != 0;
  return GN_OK;
}

gn_status gn_profile_read(gn_ctx* c, double* gemm_ms, double* gemm_flop, int64_t* gemm_launches) {
  if (!c) return GN_EINVAL;
  GN_TRY(sync(c, "profile_read"));
  double ms[5] = {0.0, 0.0, 0.0, 0.0, 0.0}, flop[5] = {0.0, 0.0, 0.0, 0.0, 0.0};
  int64_t cnt[5] = {0, 0, 0, 0, 0};
  for (size_t i = 0; i < c->ev_used; ++i) {
    float t = 0.f;
    const int k = c->ev[i].kind < 0 || c->ev[i].kind > 4 ? 1 : c->ev[i].kind;
    if (cudaEventElapsedTime(&t, c->ev[i].a, c->ev[i].b) == cudaSuccess) ms[k] += t;
    flop[k] += c->ev[i].flop;
    cnt[k] += 1;
  }
  for (int k = 0; k < 5; ++k) {
    if (gemm_ms) gemm_ms[k] = ms[k];
    if (gemm_flop) gemm_flop[k] = flop[k];
    if (gemm_launches) gemm_launches[k] = cnt[k];
  }
  c->ev_used = 0;
  cudaGetLastError();
  return GN_OK;
}

static gn_status debug_gemm_impl(gn_ctx* c, int kind, GemmArgs g);

gn_status gn_debug_gemm(gn_ctx* c, int kind, int M, int N, int K, const float* dA, int64_t lda, int a_kmajor,
                        const float* dB, int64_t ldb, int b_kmajor, float* dD, int64_t ldd) {
  return gn_debug_gemm_epilogue(c, kind, M, N, K, dA, lda, a_kmajor, dB, ldb, b_kmajor, dD, ldd, nullptr, 0, nullptr, 0,
                                1.f, nullptr, 0, 0.f);
}

gn_status gn_debug_gemm_epilogue(gn_ctx* c, int kind, int M, int N, int K, const float* dA, int64_t lda, int a_kmajor,
                                 const float* dB, int64_t ldb, int b_kmajor, float* dD, int64_t ldd, const float* d_bias,
                                 int sigmoid, const float* d_dsig, int64_t ld_dsig, float alpha, const float* d_cin,
                                 int64_t ld_cin, float beta) {
  if (!c) return GN_EINVAL;
  if (!dA || !dB || !dD || M < 1 || N < 1 || K < 1 || kind < 0 || kind > 7) return fail(c, GN_EINVAL, "bad GEMM arguments");
  if ((d_dsig && ld_dsig < N) || (d_cin && ld_cin < N)) return fail(c, GN_EINVAL, "leading dimension of an epilogue operand below N");
  GemmArgs g;
  g.M = M; g.N = N; g.K1 = K;
  g.A1 = dA; g.lda1 = lda; g.a_kmajor = a_kmajor != 0;
  g.B1 = dB; g.ldb1 = ldb; g.b_kmajor = b_kmajor != 0;
  g.D = dD; g.ldd = ldd;
  g.bias = d_bias; g.sigmoid = sigmoid != 0;
  if (d_dsig) { g.dsig = d_dsig; g.ld_dsig = ld_dsig; g.dsig_rows = M; }
  g.alpha = alpha;
  if (d_cin) { g.cin = d_cin; g.ld_cin = ld_cin; g.beta = beta; }
  return debug_gemm_impl(c, kind, g);
}

static gn_status debug_gemm_impl(gn_ctx* c, int kind, GemmArgs g) {
  // kinds 3..6 are the tensor-core kernel with options: 3 = MN-major operands declared padded,
  // 4 = one CTA per tile forced, 5 = CTA pair per tile forced, 6 = as 5 without splitting tiles
  // between pairs (all with padded operands)
  ++c->parts_epoch;
  if (kind == 7) {          // error-compensated tensor-core form (3 x TF32, chunked accumulation)
    ++c->gemm_seq;
    if (!run_gemm_x3(c, g)) return fail(c, GN_EINVAL, "the error-compensated tensor-core form does not take this problem");
    GN_TRY(check_launch(c, "debug_gemm"));
    return sync(c, "debug_gemm");
  }
  g.mn_padded = (kind >= 3);
  if (kind == 4) g.two_cta = 0;
  if (kind == 5) g.two_cta = 1;
  if (kind == 6) g.two_cta = 2;   // CTA pair per tile, whole tiles only (no stream-K split)
  if (kind >= 3) kind = 0;
  if (kind == 0 && !gemm_tf32_eligible(g)) return fail(c, GN_EINVAL, "operands do not qualify for the tensor-core kernel");
  if (kind == 2) {
    if (gemm_thin_kind(g) == THIN_NONE) return fail(c, GN_EINVAL, "operands do not qualify for a streaming kernel");
    run_gemm(c, g);
  } else {
    run_gemm_kind(c, g, kind);
  }
  GN_TRY(check_launch(c, "debug_gemm"));
  return sync(c, "debug_gemm");
}

// x^T y into device scalar slot (fixed-order double-precision sum of per-chunk partials)
static void dot_to_slot(gn_ctx* c, const float* x, const float* y, int slot) {
  c->launches += launch_cg_dot(x, y, c->chunks[0], c->n_chunks[0], c->partial, nullptr, 0, nullptr, c->st);
  c->launches += launch_sum_partials(c->partial, c->n_chunks[0], c->dscal + slot, false, c->st);
}

gn_status gn_newton_iter(gn_ctx* c, float* d_theta, const int32_t* d_idx, int64_t nS, float* d_dir,
                         const gn_newton_params* prm, gn_newton_report* rep) {
  if (!c) return GN_EINVAL;
  if (!d_theta || !d_idx || !d_dir || !prm || !rep) return fail(c, GN_EINVAL, "NULL argument");
  if (!(prm->lambda >= 0.0) || prm->cg_max < 1 || !(prm->eta > 0.0 && prm->eta < 1.0) || prm->max_backtrack < 0 ||
      !(prm->drop > 0.0) || !(prm->boost > 0.0))
    return fail(c, GN_EINVAL, "bad Newton parameters");
  for (int i = 0; i < 4; ++i)
    if (!c->nt[i]) GN_TRY(dev_alloc(c, &c->nt[i], c->n));
  float* g = c->nt[0]; float* d = c->nt[1]; float* Gx = c->nt[2]; float* trial = c->nt[3];
  const float inv_C = (float)(1.0 / c->C);
  std::memset(rep, 0, sizeof(*rep));

  GN_TRY(gn_set_theta(c, d_theta));
  GN_TRY(gn_set_subsample(c, d_idx, nS));
  double f0 = 0.0;
  GN_TRY(fun_grad(c, g, &f0));
  int its = 0;
  GN_TRY(gn_cg_solve(c, g, prm->lambda, prm->blockdiag, prm->cg_max, prm->sigma, d, &its, nullptr, nullptr));
  // entries of the two-variable system on the full G^S (Eq. sol-comp)
  GN_TRY(product_full(c, d, Gx, inv_C));
  dot_to_slot(c, d, Gx, 4);          // a  = d^T G d
  dot_to_slot(c, d_dir, Gx, 5);      // b  = dbar^T G d
  GN_TRY(product_full(c, d_dir, Gx, inv_C));
  dot_to_slot(c, d_dir, Gx, 6);      // c  = dbar^T G dbar
  dot_to_slot(c, g, d, 7);           // g^T d
  dot_to_slot(c, g, d_dir, 8);       // g^T dbar
  GN_CUDA(c, cudaMemcpyAsync(c->hscal + 4, c->dscal + 4, 5 * sizeof(double), cudaMemcpyDeviceToHost, c->st));
  GN_TRY(check_launch(c, "newton: direction combination"));
  GN_TRY(sync(c, "newton: direction combination"));
  const double a = c->hscal[4], b = c->hscal[5], cc = c->hscal[6], gd = c->hscal[7], gdb = c->hscal[8];
  double beta1 = 1.0, beta2 = 0.0;
  const double det = a * cc - b * b;
  if (det > prm->eps) { beta1 = (-gd * cc + b * gdb) / det; beta2 = (-a * gdb + b * gd) / det; }
  // d <- beta1 d + beta2 dbar, kept in d_dir (it is the next iteration's dbar)
  c->launches += launch_axpby(c->n, (float)beta1, d, (float)beta2, d_dir, d_dir, c->st);
  const double gTd = beta1 * gd + beta2 * gdb;
  const double dGd = beta1 * beta1 * a + 2.0 * beta1 * beta2 * b + beta2 * beta2 * cc;
  // back-tracking line search (Eq. linesearch-condition)
  double alpha = 1.0, f1 = 0.0;
  int backtracks = 0;
  for (;;) {
    c->launches += launch_axpby(c->n, 1.f, d_theta, (float)alpha, d_dir, trial, c->st);
    GN_TRY(gn_set_theta(c, trial));
    GN_TRY(fun_grad(c, nullptr, &f1));
    if (f1 <= f0 + prm->eta * alpha * gTd || backtracks >= prm->max_backtrack) break;
    alpha *= 0.5;
    ++backtracks;
  }
  GN_CUDA(c, cudaMemcpyAsync(d_theta, trial, c->n * sizeof(float), cudaMemcpyDeviceToDevice, c->st));
  GN_TRY(sync(c, "newton: update"));
  const double rho = (f1 - f0) / (alpha * gTd + 0.5 * alpha * alpha * dGd);
  double lam = prm->lambda;
  if (rho > 0.75) lam *= prm->drop;
  else if (!(rho >= 0.25)) lam *= prm->boost;
  rep->f_before = f0; rep->f_after = f1; rep->alpha = alpha; rep->beta1 = beta1; rep->beta2 = beta2;
  rep->rho = rho; rep->gTd = gTd; rep->dGd = dGd; rep->lambda_next = lam;
  rep->cg_iters = its; rep->backtracks = backtracks;
  return GN_OK;
}

gn_status gn_debug_option(gn_ctx* c, int option, int value) {
  if (!c) return GN_EINVAL;
  if (option == 2) { if (value < 0) return fail(c, GN_EINVAL, "count must be >= 0"); c->fail_alloc_in = value; return GN_OK; }
  if (option == 3) { quiesce(c); c->side_enabled = value != 0; return GN_OK; }
  if (option == 7) { c->split_k_enabled = value != 0; return GN_OK; }
  if (option == 8) { c->back_chain = value < 0 ? 0 : (value > 2 ? 2 : value); return GN_OK; }
  if (option == 9) { c->fly_enabled = value != 0; return GN_OK; }
  if (option == 6) { c->graph_enabled = value != 0; return GN_OK; }
  if (option == 5) { c->parts_enabled = value != 0; return GN_OK; }
  if (option == 4) { c->chain_level = value < 0 ? 0 : (value > 2 ? 2 : value); return GN_OK; }
  if (option == 0) c->group_enabled = value != 0;
  else if (option == 1) c->sk_enabled = value != 0 && c->sk_enabled;
  else return fail(c, GN_EINVAL, "unknown option");
  return GN_OK;
}

int32_t gn_debug_plan_group(int32_t n, const int32_t* M, const int32_t* N, const int32_t* K, int32_t pairs, int32_t keep_order,
                            int32_t* counts, int32_t* waves, int32_t* order, int32_t* tiles) {
  if (!M || !N || !K || !counts || !waves || !order || !tiles) return -1;
  return gemm_tf32_plan_group(n, M, N, K, pairs, keep_order, counts, waves, order, tiles);
}

gn_status gn_debug_check_canaries(gn_ctx* c, int64_t* n_checked) {
  if (!c) return GN_EINVAL;
  GN_TRY(sync(c, "canary check"));
  if (c->st2) cudaStreamSynchronize(c->st2);
  unsigned char host[128];
  int64_t checked = 0;
  for (const auto& o : c->owned) {
    if (!o.p) continue;
    GN_CUDA(c, cudaMemcpy(host, static_cast<const char*>(o.p) + o.bytes + 128, 128, cudaMemcpyDeviceToHost));
    for (int i = 0; i < 128; ++i)
      if (host[i] != kCanaryByte)
        return fail(c, GN_ECUDA, "the guard bytes after a workspace of " + std::to_string(o.bytes) + " bytes were overwritten (offset " +
                                     std::to_string(i) + " past its slack)");
    ++checked;
  }
  if (n_checked) *n_checked = checked;
  return GN_OK;
}

gn_status gn_debug_timeout_probe(gn_ctx* c, double limit_ms) {
  if (!c) return GN_EINVAL;
  if (!(limit_ms > 0.0) || limit_ms > 1000.0) return fail(c, GN_EINVAL, "limit must be in (0, 1000] ms");
  c->launches += launch_timeout_probe(c->err_flag + 1, (unsigned long long)(limit_ms * 1e6), c->st);
  GN_TRY(check_launch(c, "timeout probe"));
  return sync(c, "timeout probe");
}

gn_status gn_debug_activations(gn_ctx* c, int m, float* d_out) {
  if (!c) return GN_EINVAL;
  if (!d_out || m < 1 || m > c->L) return fail(c, GN_EINVAL, "bad layer / NULL output");
  GN_TRY(need_product_state(c));
  GN_CUDA(c, cudaMemcpyAsync(d_out, c->Z[m], c->nS * c->w[m] * sizeof(float), cudaMemcpyDeviceToDevice, c->st));
  return GN_OK;
}

}  // extern "C"
