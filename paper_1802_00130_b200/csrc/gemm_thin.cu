// Contractions with one tiny dimension (the n_L-wide output layer): memory-bound, so they run as
// streaming FP32 kernels instead of 128-wide GEMM tiles.
//
//   thin-N : D[M][N] = sum_k A[m][k] B[n][k] (+ second pair), N <= 16          (output-layer forward / R pass)
//   thin-M : D[M][N] = alpha sum_r A[r][m] B[r][n] + beta cin, M <= 16          (output-layer weight block)
//   thin-K : D[M][N] = (sum_k A[m][k] B[k][n]) * epilogue, K <= 16              (back-propagation out of layer L)
//
// All use the common epilogue of GemmArgs.  Deterministic: fixed-order reductions, no atomics.
#include <cstdio>

#include "../../include/gn.h"
#include "gn_kernels.h"

namespace gn {
namespace {

inline bool aligned16(const void* p) { return (reinterpret_cast<uintptr_t>(p) & 15) == 0; }

struct Epi {
  float* D; long long ldd;
  const float* bias; int sigmoid;
  const float* dsig; long long ld_dsig; int dsig_rows, dsig_div;
  float alpha;
  const float* cin; long long ld_cin; float beta;
};

Epi make_epi(const GemmArgs& g) {
  Epi e;
  e.D = g.D; e.ldd = g.ldd; e.bias = g.bias; e.sigmoid = g.sigmoid;
  e.dsig = g.dsig; e.ld_dsig = g.ld_dsig; e.dsig_rows = g.dsig_rows > 0 ? g.dsig_rows : 1; e.dsig_div = g.dsig_div > 0 ? g.dsig_div : 1;
  e.alpha = g.alpha; e.cin = g.cin; e.ld_cin = g.ld_cin; e.beta = g.beta;
  return e;
}

__device__ __forceinline__ float apply_epi(const Epi& e, float x, int m, int n) {
  if (e.bias) x += __ldg(e.bias + n);
  if (e.sigmoid) x = 1.f / (1.f + expf(-x));
  if (e.dsig) { const float z = __ldg(e.dsig + (long long)((m / e.dsig_div) % e.dsig_rows) * e.ld_dsig + n); x *= z * (1.f - z); }
  x *= e.alpha;
  if (e.cin) x = fmaf(e.beta, __ldg(e.cin + (long long)m * e.ld_cin + n), x);
  return x;
}

__device__ __forceinline__ float warp_sum(float v) {
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
  return v;
}

// ------------------------------------------------------------------------------------ thin-N
// One warp per group of TR rows; lanes stride K in float4 steps; B rows come through L1.
constexpr int TR = 4;

struct ThinNParams {
  int M, N;
  const float* A[2]; const float* B[2]; int K[2]; long long lda[2], ldb[2];
  Epi e;
};

template <int NMAX>
__global__ void __launch_bounds__(128, 3) gemm_thin_n_kernel(const ThinNParams p) {
  const int lane = threadIdx.x & 31;
  const int warp = blockIdx.x * (blockDim.x >> 5) + (threadIdx.x >> 5);
  const int m0 = warp * TR;
  if (m0 >= p.M) return;
  float acc[TR][NMAX];
#pragma unroll
  for (int r = 0; r < TR; ++r)
#pragma unroll
    for (int n = 0; n < NMAX; ++n) acc[r][n] = 0.f;

  for (int s = 0; s < 2; ++s) {
    const float* __restrict__ A = p.A[s];
    const float* __restrict__ B = p.B[s];
    if (!A) continue;
    const int K = p.K[s];
    const float* arow[TR];
#pragma unroll
    for (int r = 0; r < TR; ++r) arow[r] = A + (long long)min(m0 + r, p.M - 1) * p.lda[s];   // clamped rows are never written
    // software pipeline: the A rows of the next k-step are requested before this step's arithmetic
    float4 a[TR], an[TR];
    int k = lane * 4;
#pragma unroll
    for (int r = 0; r < TR; ++r) a[r] = k < K ? __ldg(reinterpret_cast<const float4*>(arow[r] + k)) : make_float4(0.f, 0.f, 0.f, 0.f);
    for (; k < K; k += 128) {
      const int kn = k + 128;
#pragma unroll
      for (int r = 0; r < TR; ++r) an[r] = kn < K ? __ldg(reinterpret_cast<const float4*>(arow[r] + kn)) : make_float4(0.f, 0.f, 0.f, 0.f);
      // all B loads of the step are issued before any of them is used: one L1 / L2 round trip per step
      // instead of one per output column (they used to serialise: 24 stall cycles per issued instruction)
      float4 b[NMAX];
#pragma unroll
      for (int n = 0; n < NMAX; ++n)
        b[n] = n < p.N ? __ldg(reinterpret_cast<const float4*>(B + (long long)n * p.ldb[s] + k)) : make_float4(0.f, 0.f, 0.f, 0.f);
#pragma unroll
      for (int n = 0; n < NMAX; ++n) {
#pragma unroll
        for (int r = 0; r < TR; ++r) {
          acc[r][n] = fmaf(a[r].x, b[n].x, acc[r][n]);
          acc[r][n] = fmaf(a[r].y, b[n].y, acc[r][n]);
          acc[r][n] = fmaf(a[r].z, b[n].z, acc[r][n]);
          acc[r][n] = fmaf(a[r].w, b[n].w, acc[r][n]);
        }
      }
#pragma unroll
      for (int r = 0; r < TR; ++r) a[r] = an[r];
    }
  }
#pragma unroll
  for (int r = 0; r < TR; ++r) {
    float mine = 0.f;
#pragma unroll
    for (int n = 0; n < NMAX; ++n) {
      const float s = warp_sum(acc[r][n]);
      if (lane == n) mine = s;
    }
    const int m = m0 + r;
    if (m < p.M && lane < p.N) p.e.D[(long long)m * p.e.ldd + lane] = apply_epi(p.e, mine, m, lane);
  }
}

// ------------------------------------------------------------------------------------ thin-M
// grid (column tiles of 512, row chunks); a thread owns 4 consecutive columns and every other row of
// the chunk; A rows staged in shared memory 128 at a time; per-chunk partials go to scratch and are
// summed in chunk order.
constexpr int TM_MAX = 16, TM_ROWS = 128;

struct ThinMParams {
  int M, N; long long rows, chunk_rows;
  const float* A; long long lda;
  const float* B; long long ldb;
  float* scratch;  // [chunks][M][N]
};

template <int MMAX>
__global__ void __launch_bounds__(256) gemm_thin_m_partial_kernel(const ThinMParams p) {
  // 256 threads = 2 row-halves x 128 column threads: half h takes rows h, h + 2, ... of the chunk, so
  // that twice as many 16-byte loads of B are in flight; the halves are added at the end.
  __shared__ __align__(16) float As[TM_ROWS][MMAX];    // (MMAX is a multiple of 4: a row is read back as 16-byte groups)
  __shared__ float4 Hs[MMAX][128];
  const int ct = threadIdx.x & 127, half = threadIdx.x >> 7;
  const int n = (blockIdx.x * 128 + ct) * 4;
  const long long r_begin = (long long)blockIdx.y * p.chunk_rows;
  const long long r_end = min(p.rows, r_begin + p.chunk_rows);
  float4 acc[MMAX];
#pragma unroll
  for (int m = 0; m < MMAX; ++m) acc[m] = make_float4(0.f, 0.f, 0.f, 0.f);
  for (long long rb = r_begin; rb < r_end; rb += TM_ROWS) {
    const int cnt = (int)min((long long)TM_ROWS, r_end - rb);
    __syncthreads();
    for (int i = threadIdx.x; i < cnt * MMAX; i += 256) {
      const int r = i / MMAX, m = i % MMAX;
      As[r][m] = m < p.M ? __ldg(p.A + (rb + r) * p.lda + m) : 0.f;
    }
    __syncthreads();
    if (n < p.N) {
#pragma unroll 8
      for (int r = half; r < cnt; r += 2) {
        const float4 b = __ldg(reinterpret_cast<const float4*>(p.B + (rb + r) * p.ldb + n));
#pragma unroll
        for (int m4 = 0; m4 < MMAX / 4; ++m4) {
          const float4 a4 = *reinterpret_cast<const float4*>(&As[r][4 * m4]);   // one shared-memory read per four rows of A
          const float av[4] = {a4.x, a4.y, a4.z, a4.w};
#pragma unroll
          for (int j = 0; j < 4; ++j) {
            const int m = 4 * m4 + j;
            acc[m].x = fmaf(av[j], b.x, acc[m].x); acc[m].y = fmaf(av[j], b.y, acc[m].y);
            acc[m].z = fmaf(av[j], b.z, acc[m].z); acc[m].w = fmaf(av[j], b.w, acc[m].w);
          }
        }
      }
    }
  }
  if (half == 1) {
#pragma unroll
    for (int m = 0; m < MMAX; ++m) Hs[m][ct] = acc[m];
  }
  __syncthreads();
  if (half == 0 && n < p.N) {
#pragma unroll
    for (int m = 0; m < MMAX; ++m)
      if (m < p.M) {
        const float4 o = Hs[m][ct];
        *reinterpret_cast<float4*>(p.scratch + ((long long)blockIdx.y * p.M + m) * p.N + n) =
            make_float4(acc[m].x + o.x, acc[m].y + o.y, acc[m].z + o.z, acc[m].w + o.w);
      }
  }
}

// One block per 32 consecutive elements of the [M][N] result (lane = element); warp w adds chunks w, w + 8, ...
// and the eight warp sums are added in warp order: a fixed order, and eight short chains instead of one long one.
__global__ void __launch_bounds__(256) gemm_thin_m_final_kernel(const float* __restrict__ scratch, int chunks, int M, int N,
                                                                const Epi e) {
  __shared__ float sh[8][33];
  const int lane = threadIdx.x & 31, w = threadIdx.x >> 5;
  const long long total = (long long)M * N;
  const long long i = (long long)blockIdx.x * 32 + lane;
  float s = 0.f;
  if (i < total)
    for (int c = w; c < chunks; c += 8) s += __ldg(scratch + (long long)c * total + i);
  sh[w][lane] = s;
  __syncthreads();
  if (w == 0 && i < total) {
    float t = sh[0][lane];
#pragma unroll
    for (int k = 1; k < 8; ++k) t += sh[k][lane];
    const int m = (int)(i / N), n = (int)(i % N);
    e.D[(long long)m * e.ldd + n] = apply_epi(e, t, m, n);
  }
}

// ------------------------------------------------------------------------------------ thin-K
// thread = 4 consecutive columns, with its K x 4 slice of B in registers; blocks walk row chunks.
constexpr int TK_MAX = 16;

struct ThinKParams {
  int M, N, K; int rows_per_block;
  const float* A; long long lda;
  const float* B; long long ldb;
  Epi e;
};

template <int KMAX>
__global__ void __launch_bounds__(128, 4) gemm_thin_k_kernel(const ThinKParams p) {
  // Rows are taken 64 at a time: their A values are staged in shared memory, then groups of 8 rows
  // first issue all their reads of the sigma' operand and only then compute and store, so
  // that 8 independent 16-byte loads per thread are in flight (a store between two loads would
  // otherwise pin their order, since D may alias the inputs as far as the compiler knows).
  constexpr int RB = 64, RG = 8;
  __shared__ __align__(16) float As[RB][KMAX];         // (KMAX is a multiple of 4: a row is read back as 16-byte groups)
  const int n = (blockIdx.x * 128 + threadIdx.x) * 4;
  const bool n_ok = n < p.N;
  float4 b[KMAX];
#pragma unroll
  for (int k = 0; k < KMAX; ++k)
    b[k] = (n_ok && k < p.K) ? __ldg(reinterpret_cast<const float4*>(p.B + (long long)k * p.ldb + n)) : make_float4(0.f, 0.f, 0.f, 0.f);
  float4 bz = make_float4(0.f, 0.f, 0.f, 0.f);
  if (p.e.bias && n_ok) bz = __ldg(reinterpret_cast<const float4*>(p.e.bias + n));
  const int m_begin = blockIdx.y * p.rows_per_block;
  const int m_end = min(p.M, m_begin + p.rows_per_block);
  for (int mb = m_begin; mb < m_end; mb += RB) {
    const int cnt = min(RB, m_end - mb);
    __syncthreads();
    for (int i = threadIdx.x; i < cnt * KMAX; i += 128) {
      const int r = i / KMAX, k = i % KMAX;
      As[r][k] = k < p.K ? __ldg(p.A + (long long)(mb + r) * p.lda + k) : 0.f;
    }
    __syncthreads();
    if (!n_ok) continue;
    for (int r0 = 0; r0 < cnt; r0 += RG) {
      float4 z[RG];
#pragma unroll
      for (int i = 0; i < RG; ++i) {
        const int m = mb + r0 + i;
        const bool ok = r0 + i < cnt;
        z[i] = (p.e.dsig && ok) ? __ldg(reinterpret_cast<const float4*>(p.e.dsig + (long long)((m / p.e.dsig_div) % p.e.dsig_rows) * p.e.ld_dsig + n))
                                : make_float4(0.f, 0.f, 0.f, 0.f);
      }
#pragma unroll
      for (int i = 0; i < RG; ++i) {
        if (r0 + i >= cnt) break;
        const int m = mb + r0 + i;
        float4 acc = bz;
#pragma unroll
        for (int k4 = 0; k4 < KMAX / 4; ++k4) {
          const float4 a4 = *reinterpret_cast<const float4*>(&As[r0 + i][4 * k4]);
          const float av[4] = {a4.x, a4.y, a4.z, a4.w};
#pragma unroll
          for (int j = 0; j < 4; ++j) {
            const int k = 4 * k4 + j;
            acc.x = fmaf(av[j], b[k].x, acc.x); acc.y = fmaf(av[j], b[k].y, acc.y);
            acc.z = fmaf(av[j], b[k].z, acc.z); acc.w = fmaf(av[j], b[k].w, acc.w);
          }
        }
        float t[4] = {acc.x, acc.y, acc.z, acc.w};
        if (p.e.sigmoid) {
#pragma unroll
          for (int j = 0; j < 4; ++j) t[j] = 1.f / (1.f + expf(-t[j]));
        }
        if (p.e.dsig) {
          t[0] *= z[i].x * (1.f - z[i].x); t[1] *= z[i].y * (1.f - z[i].y);
          t[2] *= z[i].z * (1.f - z[i].z); t[3] *= z[i].w * (1.f - z[i].w);
        }
#pragma unroll
        for (int j = 0; j < 4; ++j) t[j] *= p.e.alpha;
        if (p.e.cin) {   // not on the path's hot use of this kernel: read in place
          const float4 c = __ldg(reinterpret_cast<const float4*>(p.e.cin + (long long)m * p.e.ld_cin + n));
          t[0] = fmaf(p.e.beta, c.x, t[0]); t[1] = fmaf(p.e.beta, c.y, t[1]);
          t[2] = fmaf(p.e.beta, c.z, t[2]); t[3] = fmaf(p.e.beta, c.w, t[3]);
        }
        *reinterpret_cast<float4*>(p.e.D + (long long)m * p.e.ldd + n) = make_float4(t[0], t[1], t[2], t[3]);
      }
    }
  }
}

int thin_m_chunks(long long rows, int N) {
  const int col_tiles = (N + 511) / 512;
  long long chunks = (296 + col_tiles - 1) / col_tiles;
  const long long max_chunks = (rows + 63) / 64;
  if (chunks > max_chunks) chunks = max_chunks;
  if (chunks < 1) chunks = 1;
  return (int)chunks;
}

}  // namespace

ThinKind gemm_thin_kind(const GemmArgs& g) {
  if (g.M < 1 || g.N < 1) return THIN_NONE;
  const bool pair2 = g.A2 != nullptr;
  if (g.a_kmajor && g.b_kmajor && g.N <= 16 && g.K1 >= 64) {
    bool ok = aligned16(g.A1) && aligned16(g.B1) && g.lda1 % 4 == 0 && g.ldb1 % 4 == 0 && g.K1 % 4 == 0;
    if (pair2) ok = ok && aligned16(g.A2) && aligned16(g.B2) && g.lda2 % 4 == 0 && g.ldb2 % 4 == 0 && g.K2 % 4 == 0;
    if (ok) return THIN_N;
  }
  if (!g.a_kmajor && !g.b_kmajor && !pair2 && g.M <= TM_MAX && g.N % 4 == 0 && aligned16(g.B1) && g.ldb1 % 4 == 0)
    return THIN_M;
  if (g.a_kmajor && !g.b_kmajor && !pair2 && g.K1 <= TK_MAX && g.N % 4 == 0 && aligned16(g.B1) && g.ldb1 % 4 == 0 &&
      aligned16(g.D) && g.ldd % 4 == 0 && (!g.bias || aligned16(g.bias)) &&
      (!g.dsig || (aligned16(g.dsig) && g.ld_dsig % 4 == 0)) && (!g.cin || (aligned16(g.cin) && g.ld_cin % 4 == 0)))
    return THIN_K;
  return THIN_NONE;
}

int64_t gemm_thin_scratch_floats(const GemmArgs& g) {
  if (gemm_thin_kind(g) != THIN_M) return 0;
  return (int64_t)thin_m_chunks(g.K1, g.N) * g.M * g.N;
}

int launch_gemm_thin(const GemmArgs& g, float* scratch, cudaStream_t st) {
  const ThinKind kind = gemm_thin_kind(g);
  if (kind == THIN_N) {
    ThinNParams p{};
    p.M = g.M; p.N = g.N;
    p.A[0] = g.A1; p.B[0] = g.B1; p.K[0] = g.K1; p.lda[0] = g.lda1; p.ldb[0] = g.ldb1;
    p.A[1] = g.A2; p.B[1] = g.B2; p.K[1] = g.A2 ? g.K2 : 0; p.lda[1] = g.lda2; p.ldb[1] = g.ldb2;
    p.e = make_epi(g);
    const int warps = (g.M + TR - 1) / TR;
    const int grid = (warps + 3) / 4;
    if (g.N <= 4) gemm_thin_n_kernel<4><<<grid, 128, 0, st>>>(p);
    else if (g.N <= 8) gemm_thin_n_kernel<8><<<grid, 128, 0, st>>>(p);
    else if (g.N <= 12) gemm_thin_n_kernel<12><<<grid, 128, 0, st>>>(p);
    else gemm_thin_n_kernel<16><<<grid, 128, 0, st>>>(p);
    return 1;
  }
  if (kind == THIN_M) {
    ThinMParams p{};
    p.M = g.M; p.N = g.N; p.rows = g.K1;
    const int chunks = thin_m_chunks(g.K1, g.N);
    p.chunk_rows = (g.K1 + chunks - 1) / chunks;
    const int used = (int)((g.K1 + p.chunk_rows - 1) / p.chunk_rows);
    p.A = g.A1; p.lda = g.lda1; p.B = g.B1; p.ldb = g.ldb1; p.scratch = scratch;
    dim3 grid((g.N + 511) / 512, used);
    if (g.M <= 4) gemm_thin_m_partial_kernel<4><<<grid, 256, 0, st>>>(p);
    else if (g.M <= 8) gemm_thin_m_partial_kernel<8><<<grid, 256, 0, st>>>(p);
    else if (g.M <= 12) gemm_thin_m_partial_kernel<12><<<grid, 256, 0, st>>>(p);
    else gemm_thin_m_partial_kernel<16><<<grid, 256, 0, st>>>(p);
    const long long total = (long long)g.M * g.N;
    gemm_thin_m_final_kernel<<<(unsigned)((total + 31) / 32), 256, 0, st>>>(scratch, used, g.M, g.N, make_epi(g));
    return 2;
  }
  if (kind == THIN_K) {
    ThinKParams p{};
    p.M = g.M; p.N = g.N; p.K = g.K1;
    p.A = g.A1; p.lda = g.lda1; p.B = g.B1; p.ldb = g.ldb1; p.e = make_epi(g);
    const int col_tiles = (g.N + 511) / 512;
    int row_blocks = (148 * 8 + col_tiles - 1) / col_tiles;
    if (row_blocks > g.M) row_blocks = g.M;
    p.rows_per_block = (g.M + row_blocks - 1) / row_blocks;
    dim3 grid(col_tiles, (g.M + p.rows_per_block - 1) / p.rows_per_block);
    if (g.K1 <= 4) gemm_thin_k_kernel<4><<<grid, 128, 0, st>>>(p);
    else if (g.K1 <= 8) gemm_thin_k_kernel<8><<<grid, 128, 0, st>>>(p);
    else if (g.K1 <= 12) gemm_thin_k_kernel<12><<<grid, 128, 0, st>>>(p);
    else gemm_thin_k_kernel<16><<<grid, 128, 0, st>>>(p);
    return 1;
  }
  return 0;
}

}  // namespace gn

// ------------------------------------------------------------------------------------ allocation-free thin-M entry
// Scratch for gn_thin_m_gemm_noalloc: a fixed array inside the library image instead of a buffer from
// cudaMalloc.  Every device that loads the library carries these 8 MiB until the process exits.
namespace {
constexpr long long kNoAllocScratchFloats = 2097152;   // 8 MiB
static __device__ __align__(256) float g_noalloc_scratch[kNoAllocScratchFloats];

constexpr int kMaxDevices = 64;
float* g_noalloc_ptr[kMaxDevices] = {};   // device address of the array, looked up once per device

void put_msg(char* buf, int64_t len, const char* msg) {
  if (buf && len > 0) snprintf(buf, (size_t)len, "%s", msg);
}
}  // namespace

extern "C" gn_status gn_thin_m_gemm_noalloc(int M, int N, int64_t rows, const float* dA, int64_t lda, const float* dB,
                                            int64_t ldb, float* dD, int64_t ldd, void* cuda_stream, char* errbuf,
                                            int64_t errbuf_len) {
  using namespace gn;
  if (!dA || !dB || !dD || M < 1 || N < 1 || rows < 1 || lda < M || ldb < N || ldd < N) {
    put_msg(errbuf, errbuf_len, "null pointer, non-positive size, or leading dimension smaller than the row length");
    return GN_EINVAL;
  }
  if (rows > 0x7fffffffLL) { put_msg(errbuf, errbuf_len, "rows exceeds 2^31 - 1"); return GN_EINVAL; }
  GemmArgs g;
  g.M = M; g.N = N; g.K1 = (int)rows;
  g.A1 = dA; g.lda1 = lda; g.a_kmajor = false;
  g.B1 = dB; g.ldb1 = ldb; g.b_kmajor = false;
  g.D = dD; g.ldd = ldd;
  if (gemm_thin_kind(g) != THIN_M) {
    put_msg(errbuf, errbuf_len, "shape not taken: needs M <= 16, N a multiple of 4, B 16-byte aligned with ldb a multiple of 4");
    return GN_EINVAL;
  }
  const long long need = gemm_thin_scratch_floats(g);
  if (need > kNoAllocScratchFloats) {
    char msg[200];
    snprintf(msg, sizeof msg, "problem needs %lld scratch floats (row chunks x M x N); the built-in scratch holds %lld",
             need, kNoAllocScratchFloats);
    put_msg(errbuf, errbuf_len, msg);
    return GN_EINVAL;
  }
  int dev = -1;
  if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= kMaxDevices) {
    cudaGetLastError();
    put_msg(errbuf, errbuf_len, "no current CUDA device (or device ordinal >= 64)");
    return GN_ECUDA;
  }
  if (!g_noalloc_ptr[dev]) {
    // In host code the array's name is only a handle; the kernels need its address on this device.
    float* ptr = nullptr;
    const cudaError_t e = cudaGetSymbolAddress(reinterpret_cast<void**>(&ptr), g_noalloc_scratch);
    if (e != cudaSuccess || !ptr) {
      cudaGetLastError();
      put_msg(errbuf, errbuf_len, cudaGetErrorString(e));
      return GN_ECUDA;
    }
    g_noalloc_ptr[dev] = ptr;
  }
  launch_gemm_thin(g, g_noalloc_ptr[dev], static_cast<cudaStream_t>(cuda_stream));
  const cudaError_t e = cudaGetLastError();
  if (e != cudaSuccess) { put_msg(errbuf, errbuf_len, cudaGetErrorString(e)); return GN_ECUDA; }
  put_msg(errbuf, errbuf_len, "");
  return GN_OK;
}
