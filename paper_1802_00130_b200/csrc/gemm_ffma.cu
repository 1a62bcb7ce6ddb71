// FP32 fused-multiply-add GEMM with the fused epilogues of the Gauss-Newton product path.
//
// Used for every contraction in GN_FP32_ACCURATE mode and, in GN_TF32 mode, for the shapes the
// tensor-core kernel does not take (n_L-wide output-layer products, unaligned operands).
//
// 128 x 128 x 16 tiles, 256 threads, 8 x 8 accumulators per thread, double-buffered shared memory
// with the next tile's global loads in flight during the current tile's arithmetic.
#include "gn_kernels.h"

namespace gn {
namespace {

constexpr int BM = 128, BN = 128, BK = 16, NT = 256, PAD = 4;

struct FfmaParams {
  int M, N;
  const float* A[2]; const float* B[2]; int K[2]; long long lda[2], ldb[2];
  int vecA[2], vecB[2];
  float* D; long long ldd;
  const float* bias; int sigmoid;
  const float* dsig; long long ld_dsig; int dsig_rows, dsig_div;
  float alpha;
  const float* cin; long long ld_cin; float beta;
  int vec_epi;
};

// Four consecutive elements along the contiguous dimension `c` of a matrix whose other index is `r`.
__device__ __forceinline__ float4 load4(const float* __restrict__ base, long long ld, int r, int c, int R,
                                        int Cn, bool vec) {
  float4 v = make_float4(0.f, 0.f, 0.f, 0.f);
  if (r >= R || c >= Cn) return v;
  const float* p = base + (long long)r * ld + c;
  if (vec && c + 3 < Cn) {
    v = __ldg(reinterpret_cast<const float4*>(p));
  } else {
    v.x = __ldg(p);
    if (c + 1 < Cn) v.y = __ldg(p + 1);
    if (c + 2 < Cn) v.z = __ldg(p + 2);
    if (c + 3 < Cn) v.w = __ldg(p + 3);
  }
  return v;
}

template <bool A_KMAJOR, bool B_KMAJOR>
__global__ void __launch_bounds__(NT, 2) gemm_ffma_kernel(const FfmaParams p) {
  __shared__ __align__(16) float As[2][BK][BM + PAD];
  __shared__ __align__(16) float Bs[2][BK][BN + PAD];

  const int tid = threadIdx.x;
  const int tx = tid & 15, ty = tid >> 4;
  const int m0 = blockIdx.y * BM, n0 = blockIdx.x * BN;

  const int nk0 = (p.K[0] + BK - 1) / BK;
  const int nk1 = p.A[1] ? (p.K[1] + BK - 1) / BK : 0;
  const int nk = nk0 + nk1;

  float acc[8][8];
#pragma unroll
  for (int i = 0; i < 8; ++i)
#pragma unroll
    for (int j = 0; j < 8; ++j) acc[i][j] = 0.f;

  float4 ra[2], rb[2];

  auto fetch = [&](int kt) {
    const int s = kt < nk0 ? 0 : 1;
    const int k0 = (s == 0 ? kt : kt - nk0) * BK;
    const float* A = p.A[s];
    const float* B = p.B[s];
    const int K = p.K[s];
#pragma unroll
    for (int i = 0; i < 2; ++i) {
      const int idx = tid + i * NT;
      if (A_KMAJOR) ra[i] = load4(A, p.lda[s], m0 + (idx >> 2), k0 + (idx & 3) * 4, p.M, K, p.vecA[s]);
      else          ra[i] = load4(A, p.lda[s], k0 + (idx >> 5), m0 + (idx & 31) * 4, K, p.M, p.vecA[s]);
      if (B_KMAJOR) rb[i] = load4(B, p.ldb[s], n0 + (idx >> 2), k0 + (idx & 3) * 4, p.N, K, p.vecB[s]);
      else          rb[i] = load4(B, p.ldb[s], k0 + (idx >> 5), n0 + (idx & 31) * 4, K, p.N, p.vecB[s]);
    }
  };
  auto stash = [&](int buf) {
#pragma unroll
    for (int i = 0; i < 2; ++i) {
      const int idx = tid + i * NT;
      if (A_KMAJOR) {
        const int r = idx >> 2, kq = (idx & 3) * 4;
        As[buf][kq + 0][r] = ra[i].x; As[buf][kq + 1][r] = ra[i].y;
        As[buf][kq + 2][r] = ra[i].z; As[buf][kq + 3][r] = ra[i].w;
      } else {
        *reinterpret_cast<float4*>(&As[buf][idx >> 5][(idx & 31) * 4]) = ra[i];
      }
      if (B_KMAJOR) {
        const int r = idx >> 2, kq = (idx & 3) * 4;
        Bs[buf][kq + 0][r] = rb[i].x; Bs[buf][kq + 1][r] = rb[i].y;
        Bs[buf][kq + 2][r] = rb[i].z; Bs[buf][kq + 3][r] = rb[i].w;
      } else {
        *reinterpret_cast<float4*>(&Bs[buf][idx >> 5][(idx & 31) * 4]) = rb[i];
      }
    }
  };

  if (nk > 0) {
    fetch(0);
    stash(0);
  }
  __syncthreads();

  int cur = 0;
  for (int kt = 0; kt < nk; ++kt) {
    if (kt + 1 < nk) fetch(kt + 1);
#pragma unroll
    for (int k = 0; k < BK; ++k) {
      const float4 a0 = *reinterpret_cast<const float4*>(&As[cur][k][ty * 4]);
      const float4 a1 = *reinterpret_cast<const float4*>(&As[cur][k][64 + ty * 4]);
      const float4 b0 = *reinterpret_cast<const float4*>(&Bs[cur][k][tx * 4]);
      const float4 b1 = *reinterpret_cast<const float4*>(&Bs[cur][k][64 + tx * 4]);
      const float a[8] = {a0.x, a0.y, a0.z, a0.w, a1.x, a1.y, a1.z, a1.w};
      const float b[8] = {b0.x, b0.y, b0.z, b0.w, b1.x, b1.y, b1.z, b1.w};
#pragma unroll
      for (int i = 0; i < 8; ++i)
#pragma unroll
        for (int j = 0; j < 8; ++j) acc[i][j] = fmaf(a[i], b[j], acc[i][j]);
    }
    if (kt + 1 < nk) {
      stash(cur ^ 1);
      __syncthreads();
      cur ^= 1;
    }
  }

  // ---- epilogue
#pragma unroll
  for (int i = 0; i < 8; ++i) {
    const int m = m0 + (i < 4 ? ty * 4 + i : 64 + ty * 4 + (i - 4));
    if (m >= p.M) continue;
    const long long zrow = p.dsig ? (long long)((m / p.dsig_div) % p.dsig_rows) * p.ld_dsig : 0;
#pragma unroll
    for (int h = 0; h < 2; ++h) {
      const int n = n0 + h * 64 + tx * 4;
      if (n >= p.N) continue;
      float t[4] = {acc[i][h * 4 + 0], acc[i][h * 4 + 1], acc[i][h * 4 + 2], acc[i][h * 4 + 3]};
      const bool v4 = p.vec_epi && (n + 3 < p.N);
      const int cnt = min(4, p.N - n);
      float bz[4] = {0.f, 0.f, 0.f, 0.f}, zc[4] = {0.f, 0.f, 0.f, 0.f}, ci[4] = {0.f, 0.f, 0.f, 0.f};
      if (v4) {
        if (p.bias) { const float4 x = __ldg(reinterpret_cast<const float4*>(p.bias + n)); bz[0] = x.x; bz[1] = x.y; bz[2] = x.z; bz[3] = x.w; }
        if (p.dsig) { const float4 x = __ldg(reinterpret_cast<const float4*>(p.dsig + zrow + n)); zc[0] = x.x; zc[1] = x.y; zc[2] = x.z; zc[3] = x.w; }
        if (p.cin)  { const float4 x = __ldg(reinterpret_cast<const float4*>(p.cin + (long long)m * p.ld_cin + n)); ci[0] = x.x; ci[1] = x.y; ci[2] = x.z; ci[3] = x.w; }
      } else {
        for (int j = 0; j < cnt; ++j) {
          if (p.bias) bz[j] = __ldg(p.bias + n + j);
          if (p.dsig) zc[j] = __ldg(p.dsig + zrow + n + j);
          if (p.cin)  ci[j] = __ldg(p.cin + (long long)m * p.ld_cin + n + j);
        }
      }
#pragma unroll
      for (int j = 0; j < 4; ++j) {
        float x = t[j] + bz[j];
        if (p.sigmoid) x = 1.f / (1.f + expf(-x));
        if (p.dsig) x *= zc[j] * (1.f - zc[j]);
        x *= p.alpha;
        if (p.cin) x = fmaf(p.beta, ci[j], x);
        t[j] = x;
      }
      float* dp = p.D + (long long)m * p.ldd + n;
      if (v4) {
        *reinterpret_cast<float4*>(dp) = make_float4(t[0], t[1], t[2], t[3]);
      } else {
        for (int j = 0; j < cnt; ++j) dp[j] = t[j];
      }
    }
  }
}

inline bool aligned16(const void* p) { return (reinterpret_cast<uintptr_t>(p) & 15) == 0; }

}  // namespace

int launch_gemm_ffma(const GemmArgs& g, cudaStream_t st) {
  if (g.M <= 0 || g.N <= 0) return 0;
  FfmaParams p{};
  p.M = g.M; p.N = g.N;
  p.A[0] = g.A1; p.B[0] = g.B1; p.K[0] = g.K1; p.lda[0] = g.lda1; p.ldb[0] = g.ldb1;
  p.A[1] = g.A2; p.B[1] = g.B2; p.K[1] = g.A2 ? g.K2 : 0; p.lda[1] = g.lda2; p.ldb[1] = g.ldb2;
  for (int s = 0; s < 2; ++s) {
    p.vecA[s] = p.A[s] && aligned16(p.A[s]) && (p.lda[s] % 4 == 0);
    p.vecB[s] = p.B[s] && aligned16(p.B[s]) && (p.ldb[s] % 4 == 0);
  }
  p.D = g.D; p.ldd = g.ldd;
  p.bias = g.bias; p.sigmoid = g.sigmoid;
  p.dsig = g.dsig; p.ld_dsig = g.ld_dsig; p.dsig_rows = g.dsig_rows > 0 ? g.dsig_rows : 1; p.dsig_div = g.dsig_div > 0 ? g.dsig_div : 1;
  p.alpha = g.alpha;
  p.cin = g.cin; p.ld_cin = g.ld_cin; p.beta = g.beta;
  p.vec_epi = aligned16(g.D) && (g.ldd % 4 == 0) && (!g.bias || aligned16(g.bias)) &&
              (!g.dsig || (aligned16(g.dsig) && g.ld_dsig % 4 == 0)) &&
              (!g.cin || (aligned16(g.cin) && g.ld_cin % 4 == 0));
  dim3 grid((g.N + BN - 1) / BN, (g.M + BM - 1) / BM);
  if (g.a_kmajor && g.b_kmajor)        gemm_ffma_kernel<true, true><<<grid, NT, 0, st>>>(p);
  else if (g.a_kmajor && !g.b_kmajor)  gemm_ffma_kernel<true, false><<<grid, NT, 0, st>>>(p);
  else if (!g.a_kmajor && g.b_kmajor)  gemm_ffma_kernel<false, true><<<grid, NT, 0, st>>>(p);
  else                                 gemm_ffma_kernel<false, false><<<grid, NT, 0, st>>>(p);
  return 1;
}

}  // namespace gn
