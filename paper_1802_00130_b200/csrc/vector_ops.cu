// Memory-bound kernels of the path: subsample row gather, column sums (bias blocks), squared loss,
// and the conjugate-gradient vector updates with their dot products.
//
// Reductions are deterministic: every block writes one partial, partials are combined in a fixed
// order in double precision.
#include <initializer_list>

#include "gn_kernels.h"

namespace gn {
namespace {

__device__ __forceinline__ double warp_sum(double v) {
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
  return v;
}
__device__ __forceinline__ float warp_sum(float v) {
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
  return v;
}

// Sum over a 256-thread block; result valid in thread 0.
__device__ __forceinline__ double block_sum_256(double v) {
  __shared__ double sh[8];
  v = warp_sum(v);
  const int w = threadIdx.x >> 5, l = threadIdx.x & 31;
  __syncthreads();
  if (l == 0) sh[w] = v;
  __syncthreads();
  double t = 0.0;
  if (w == 0) {
    t = l < 8 ? sh[l] : 0.0;
    t = warp_sum(t);
  }
  return t;
}

// ---------------------------------------------------------------------------------- gather
// One warp per destination row, 16-byte loads when the rows allow it.
__global__ void __launch_bounds__(256) gather_rows_kernel(const float* __restrict__ src, long long src_rows, int cols,
                                                          const int32_t* __restrict__ idx, long long n_idx,
                                                          float* __restrict__ dst, int* err_flag, int vec) {
  const int lane = threadIdx.x & 31;
  const long long warps = (long long)gridDim.x * (blockDim.x >> 5);
  for (long long r = (long long)blockIdx.x * (blockDim.x >> 5) + (threadIdx.x >> 5); r < n_idx; r += warps) {
    const long long s = idx[r];
    const bool ok = s >= 0 && s < src_rows;
    if (!ok && lane == 0) atomicExch(err_flag, 1);
    float* d = dst + r * cols;
    if (vec) {
      const float4* sp = reinterpret_cast<const float4*>(src + (ok ? s : 0) * cols);
      float4* dp = reinterpret_cast<float4*>(d);
      for (int c = lane; c < (cols >> 2); c += 32) dp[c] = ok ? __ldg(sp + c) : make_float4(0.f, 0.f, 0.f, 0.f);
    } else {
      const float* sp = src + (ok ? s : 0) * cols;
      for (int c = lane; c < cols; c += 32) d[c] = ok ? __ldg(sp + c) : 0.f;
    }
  }
}

// ---------------------------------------------------------------------------------- column sums
constexpr int CS_ROWS = 256;  // rows per block

// Scalar version (any alignment): grid (ceil(cols/32), ceil(rows/CS_ROWS)); 8 warps stride rows.
__global__ void __launch_bounds__(256) colsum_partial_kernel(const float* __restrict__ A, long long rows, int cols,
                                                             long long lda, float* __restrict__ scratch) {
  __shared__ float sh[8][33];
  const int lane = threadIdx.x & 31, w = threadIdx.x >> 5;
  const int c = blockIdx.x * 32 + lane;
  const long long r0 = (long long)blockIdx.y * CS_ROWS;
  const long long r1 = min(rows, r0 + CS_ROWS);
  float s = 0.f;
  if (c < cols)
    for (long long r = r0 + w; r < r1; r += 8) s += __ldg(A + r * lda + c);
  sh[w][lane] = s;
  __syncthreads();
  if (w == 0) {
    float t = 0.f;
#pragma unroll
    for (int k = 0; k < 8; ++k) t += sh[k][lane];
    if (c < cols) scratch[(long long)blockIdx.y * cols + c] = t;
  }
}

// 16-byte version: grid (ceil(cols/128), ceil(rows/CS_ROWS)); a warp covers 128 columns of a row,
// 8 warps stride rows with four rows in flight per thread.  Held to 40 registers so that a block fits on an SM
// beside a CTA of the tensor-core kernel (320 threads x 168 registers): the sums run on a side stream under it.
__global__ void __launch_bounds__(256, 6) colsum_partial_vec_kernel(const float* __restrict__ A, long long rows, int cols,
                                                                 long long lda, float* __restrict__ scratch) {
  __shared__ float4 sh[8][32];
  const int lane = threadIdx.x & 31, w = threadIdx.x >> 5;
  const int c = (blockIdx.x * 32 + lane) * 4;
  const long long r0 = (long long)blockIdx.y * CS_ROWS;
  const long long r1 = min(rows, r0 + CS_ROWS);
  float4 s = make_float4(0.f, 0.f, 0.f, 0.f);
  if (c < cols) {
    long long r = r0 + w;
    const float4* ptr = reinterpret_cast<const float4*>(A + r * lda + c);
    const long long step = 2 * lda;                       // eight rows, in 16-byte units
    for (; r + 24 < r1; r += 32, ptr += 4 * step) {
      const float4 x0 = __ldg(ptr);
      const float4 x1 = __ldg(ptr + step);
      const float4 x2 = __ldg(ptr + 2 * step);
      const float4 x3 = __ldg(ptr + 3 * step);
      s.x += (x0.x + x1.x) + (x2.x + x3.x); s.y += (x0.y + x1.y) + (x2.y + x3.y);
      s.z += (x0.z + x1.z) + (x2.z + x3.z); s.w += (x0.w + x1.w) + (x2.w + x3.w);
    }
    for (; r < r1; r += 8, ptr += step) {
      const float4 x = __ldg(ptr);
      s.x += x.x; s.y += x.y; s.z += x.z; s.w += x.w;
    }
  }
  sh[w][lane] = s;
  __syncthreads();
  if (w == 0 && c < cols) {
    float4 t = sh[0][lane];
#pragma unroll
    for (int k = 1; k < 8; ++k) { t.x += sh[k][lane].x; t.y += sh[k][lane].y; t.z += sh[k][lane].z; t.w += sh[k][lane].w; }
    *reinterpret_cast<float4*>(scratch + (long long)blockIdx.y * cols + c) = t;
  }
}

// One block per 32 columns (lane = column); warp w adds parts w, w + 8, ... and the eight warp sums are added
// in warp order.  Double precision, fixed order; eight short chains instead of one long one per column.
__global__ void __launch_bounds__(256) colsum_final_kernel(const float* __restrict__ scratch, int n_parts, int cols,
                                                           float alpha, const float* __restrict__ cin, float beta,
                                                           float* __restrict__ out) {
  __shared__ double sh[8][33];
  const int lane = threadIdx.x & 31, w = threadIdx.x >> 5;
  const int c = blockIdx.x * 32 + lane;
  double s = 0.0;
  if (c < cols)
    for (int k = w; k < n_parts; k += 8) s += (double)__ldg(scratch + (long long)k * cols + c);
  sh[w][lane] = s;
  __syncthreads();
  if (w == 0 && c < cols) {
    double t = sh[0][lane];
#pragma unroll
    for (int k = 1; k < 8; ++k) t += sh[k][lane];
    float v = alpha * (float)t;
    if (cin) v = fmaf(beta, cin[c], v);
    out[c] = v;
  }
}

// ---------------------------------------------------------------------------------- loss
constexpr int LOSS_PER_BLOCK = 256 * 8;

__global__ void __launch_bounds__(256) loss_delta_kernel(const float* __restrict__ Z, const float* __restrict__ Y,
                                                         long long count, float* __restrict__ delta,
                                                         double* __restrict__ partial) {
  const long long base = (long long)blockIdx.x * LOSS_PER_BLOCK;
  float s = 0.f;
#pragma unroll
  for (int k = 0; k < 8; ++k) {
    const long long i = base + k * 256 + threadIdx.x;
    if (i < count) {
      const float e = Z[i] - __ldg(Y + i);
      s = fmaf(e, e, s);
      if (delta) delta[i] = 2.f * e;
    }
  }
  const double t = block_sum_256((double)s);
  if (threadIdx.x == 0) partial[blockIdx.x] = t;
}

__global__ void __launch_bounds__(256) sum_partials_kernel(const double* __restrict__ partial, int count,
                                                           double* out, int accumulate) {
  double s = 0.0;
  for (int i = threadIdx.x; i < count; i += 256) s += partial[i];
  const double t = block_sum_256(s);
  if (threadIdx.x == 0) *out = accumulate ? *out + t : t;
}

// ---------------------------------------------------------------------------------- out = a x + b y
__global__ void __launch_bounds__(256) axpby_kernel(long long n, float a, const float* x, float b, const float* y,
                                                    float* out) {
  // out may be x or y (same index read and written by the same thread)
  for (long long i = (long long)blockIdx.x * 256 + threadIdx.x; i < n; i += (long long)gridDim.x * 256)
    out[i] = fmaf(a, x[i], b * y[i]);
}

// ---------------------------------------------------------------------------------- stored Jacobian factors
// D[(i, u)][t] = WL[u][t] * z (1 - z): one block per sample row i, threads over t (16-byte accesses when n % 4 == 0).
__global__ void __launch_bounds__(256) factor_last_kernel(const float* __restrict__ WL, const float* __restrict__ Zprev,
                                                          int nL, int n, float* __restrict__ D) {
  const long long i = blockIdx.x;
  const float* z = Zprev + i * n;
  float* d = D + i * nL * n;
  for (int t = threadIdx.x; t < n; t += 256) {
    const float zz = __ldg(z + t);
    const float ds = zz * (1.f - zz);
    for (int u = 0; u < nL; ++u) d[(long long)u * n + t] = __ldg(WL + (long long)u * n + t) * ds;
  }
}

// One block per (sample row i, neuron group b of the layer): the group's columns [col0, col1) of D_i are the
// factor of every partition (T_{m-1}, T_m = group b); `streams` right-hand sides (one per group of layer m-1),
// `stream_stride` floats apart in U and Q, share them.  Pass 1 forms p_u = D_i[u][T_b] . U_i[T_b] (block
// reduction per u), pass 2 re-reads D_i (just read, so from cache) and writes Q_i[j] = 2 sum_u D_i[u][j] p_u.
// NLMAX bounds n_L.  With groups = 1 and streams = 1 this is the product of a whole layer block.
template <int NLMAX>
__global__ void __launch_bounds__(256) factor_apply_kernel(const float* __restrict__ D, const float* __restrict__ U,
                                                           int nL, int n, int groups, int streams, long long stream_stride,
                                                           float* __restrict__ Q) {
  __shared__ float red[8][NLMAX];
  __shared__ float pu[NLMAX];
  const long long i = blockIdx.x;
  const int col0 = (int)(((long long)blockIdx.y * n) / groups), col1 = (int)(((long long)(blockIdx.y + 1) * n) / groups);
  const float* d = D + i * nL * n;
  const int lane = threadIdx.x & 31, w = threadIdx.x >> 5;
  for (int a = 0; a < streams; ++a) {
    const float* u_row = U + a * stream_stride + i * n;
    float* q_row = Q + a * stream_stride + i * n;
    float acc[NLMAX];
#pragma unroll
    for (int u = 0; u < NLMAX; ++u) acc[u] = 0.f;
    for (int j = col0 + threadIdx.x; j < col1; j += 256) {
      const float uj = __ldg(u_row + j);
#pragma unroll
      for (int u = 0; u < NLMAX; ++u)
        if (u < nL) acc[u] = fmaf(__ldg(d + (long long)u * n + j), uj, acc[u]);
    }
#pragma unroll
    for (int u = 0; u < NLMAX; ++u) {
      const float s = warp_sum(acc[u]);
      if (lane == 0) red[w][u] = s;
    }
    __syncthreads();
    if (threadIdx.x < NLMAX) {
      float s = 0.f;
#pragma unroll
      for (int k = 0; k < 8; ++k) s += red[k][threadIdx.x];
      pu[threadIdx.x] = 2.f * s;                              // B = 2I
    }
    __syncthreads();
    for (int j = col0 + threadIdx.x; j < col1; j += 256) {
      float q = 0.f;
#pragma unroll
      for (int u = 0; u < NLMAX; ++u)
        if (u < nL) q = fmaf(__ldg(d + (long long)u * n + j), pu[u], q);
      q_row[j] = q;
    }
  }
}

// ---------------------------------------------------------------------------------- CG
// One block per chunk of at most kCgChunk coordinates (256 threads; 16-byte accesses when the chunk starts on a
// multiple of four coordinates).  A kernel that ends in a dot product also computes the step's scalars: every
// block leaves its partial sum, takes a ticket, and the block that draws the last ticket adds the partials of every
// segment in a fixed order (so the result does not depend on which block that is) and updates the per-segment
// scalars; no separate launch, no wait.

// Per-segment sums of the chunk partials and the scalar updates of one phase, by one 256-thread block.
// phase 0: rho = gnorm2 = sum, active = rho > 0
// phase 1: pq = sum, alpha = active ? rho / pq : 0
// phase 2: rho_new = sum; beta = rho_new / rho; rho = rho_new; active &= !(stop rule met)
// ctl->out[0] = sum over segments of rho, ctl->out[1] = number of active segments; after phases 0 and 2 the
// residual norm squared is appended to the history, and a step that began with an active segment is counted.
__device__ void cg_scalars_block(int phase, const double* partial, CgSeg* seg, int n_seg, double tol, CgControl* ctl) {
  __shared__ double seg_rho[64];
  __shared__ int seg_act[64];
  __shared__ int was_active;
  const int lane = threadIdx.x & 31, w = threadIdx.x >> 5;
  if (threadIdx.x == 0) was_active = 0;
  __syncthreads();
  auto update = [&](int s, double acc) -> CgSeg {
    CgSeg g = seg[s];
    if (phase == 0) {
      g.rho = acc; g.gnorm2 = acc; g.pq = 0.0; g.alpha = 0.f; g.beta = 0.f;
      g.active = (acc > 0.0) && (tol <= 0.0 || sqrt(acc) > tol * sqrt(acc)) ? 1 : 0;
    } else if (phase == 1) {
      g.pq = acc;
      g.alpha = (g.active && acc > 0.0) ? (float)(g.rho / acc) : 0.f;
      if (!(acc > 0.0)) g.active = 0;
    } else {
      if (g.active) {
        was_active = 1;
        g.beta = g.rho > 0.0 ? (float)(acc / g.rho) : 0.f;
        g.rho = acc;
        if (!(acc > 0.0) || (tol > 0.0 && sqrt(acc) <= tol * sqrt(g.gnorm2))) g.active = 0;
      } else {
        g.beta = 0.f; g.alpha = 0.f;
      }
    }
    seg[s] = g;
    return g;
  };
  double tot = 0.0, act = 0.0;
  if (n_seg == 1) {
    const int first = seg[0].first, count = seg[0].count;
    double acc = 0.0;
    for (int c = threadIdx.x; c < count; c += 256) acc += __ldcg(partial + first + c);
    acc = block_sum_256(acc);
    if (threadIdx.x == 0) {
      const CgSeg g = update(0, acc);
      tot = g.rho; act = (double)g.active;
    }
  } else {
    for (int s0 = 0; s0 < n_seg; s0 += 64) {
      for (int s = s0 + w; s < min(n_seg, s0 + 64); s += 8) {
        const int first = seg[s].first, count = seg[s].count;
        double acc = 0.0;
        for (int c = lane; c < count; c += 32) acc += __ldcg(partial + first + c);
        acc = warp_sum(acc);
        if (lane == 0) {
          const CgSeg g = update(s, acc);
          seg_rho[s - s0] = g.rho;
          seg_act[s - s0] = g.active;
        }
      }
      __syncthreads();
      if (threadIdx.x == 0)
        for (int s = s0; s < min(n_seg, s0 + 64); ++s) { tot += seg_rho[s - s0]; act += seg_act[s - s0]; }
      __syncthreads();
    }
  }
  __syncthreads();
  if (threadIdx.x == 0) {
    ctl->out[0] = tot; ctl->out[1] = act;
    if (phase == 0) { ctl->steps = 0; ctl->hist_len = 0; }
    if (phase == 2 && was_active) ctl->steps += 1;
    if (phase != 1 && ctl->hist && ctl->hist_len < ctl->hist_cap && (phase == 0 || was_active)) ctl->hist[ctl->hist_len++] = tot;
  }
}

// Block-wide: leave this block's partial, and tell whether this block drew the last ticket of the launch.
__device__ __forceinline__ bool cg_last_block(double block_total, double* partial, CgControl* ctl) {
  __shared__ int last;
  if (threadIdx.x == 0) {
    partial[blockIdx.x] = block_total;
    __threadfence();
    const unsigned t = atomicAdd(&ctl->ticket, 1u);
    last = (t == gridDim.x - 1) ? 1 : 0;
    if (last) { ctl->ticket = 0; __threadfence(); }
  }
  __syncthreads();
  return last != 0;
}

template <typename F>
__device__ __forceinline__ void cg_for_chunk(const CgChunk& ch, bool vec_ok, F&& body4, int& tail0) {
  // body4(k) handles coordinates k .. k + 3 as one 16-byte access; the rest is left to the caller from tail0 on
  tail0 = 0;
  if (vec_ok && (ch.start & 3) == 0) {
    const int n4 = ch.len >> 2;
    for (int i = threadIdx.x; i < n4; i += 256) body4(ch.start + 4ll * i);
    tail0 = n4 << 2;
  }
}

__global__ void __launch_bounds__(256) cg_init_kernel(const float* __restrict__ g, float* __restrict__ d,
                                                      float* __restrict__ r, float* __restrict__ p,
                                                      const CgChunk* __restrict__ chunks, double* __restrict__ partial,
                                                      CgSeg* seg, int n_seg, double tol, CgControl* ctl, int vec_ok) {
  const CgChunk ch = chunks[blockIdx.x];
  float s = 0.f;
  int t0;
  cg_for_chunk(ch, vec_ok != 0, [&](long long k) {
    float4 x = *reinterpret_cast<const float4*>(g + k);
    x.x = -x.x; x.y = -x.y; x.z = -x.z; x.w = -x.w;
    *reinterpret_cast<float4*>(d + k) = make_float4(0.f, 0.f, 0.f, 0.f);
    *reinterpret_cast<float4*>(r + k) = x;
    *reinterpret_cast<float4*>(p + k) = x;
    s += x.x * x.x + x.y * x.y + x.z * x.z + x.w * x.w;
  }, t0);
  for (int i = t0 + threadIdx.x; i < ch.len; i += 256) {
    const long long k = ch.start + i;
    const float x = -g[k];
    d[k] = 0.f; r[k] = x; p[k] = x;
    s = fmaf(x, x, s);
  }
  const double t = block_sum_256((double)s);
  if (cg_last_block(t, partial, ctl)) cg_scalars_block(0, partial, seg, n_seg, tol, ctl);
}

// partial[c] = sum x y over chunk c; with seg != nullptr also the phase-1 scalars (alpha) by the last block
__global__ void __launch_bounds__(256) cg_dot_kernel(const float* __restrict__ x, const float* __restrict__ y,
                                                     const CgChunk* __restrict__ chunks, double* __restrict__ partial,
                                                     CgSeg* seg, int n_seg, CgControl* ctl, int vec_ok) {
  const CgChunk ch = chunks[blockIdx.x];
  float s = 0.f;
  int t0;
  cg_for_chunk(ch, vec_ok != 0, [&](long long k) {
    const float4 a = *reinterpret_cast<const float4*>(x + k);
    const float4 b = *reinterpret_cast<const float4*>(y + k);
    s += a.x * b.x + a.y * b.y + a.z * b.z + a.w * b.w;
  }, t0);
  for (int i = t0 + threadIdx.x; i < ch.len; i += 256) {
    const long long k = ch.start + i;
    s = fmaf(x[k], y[k], s);
  }
  const double t = block_sum_256((double)s);
  if (!seg) {
    if (threadIdx.x == 0) partial[blockIdx.x] = t;
    return;
  }
  if (cg_last_block(t, partial, ctl)) cg_scalars_block(1, partial, seg, n_seg, 0.0, ctl);
}

// d += alpha p, r -= alpha q for the live segments, partial = sum r^2, then the phase-2 scalars by the last block
__global__ void __launch_bounds__(256) cg_update_kernel(const float* __restrict__ p, const float* __restrict__ q,
                                                        float* __restrict__ d, float* __restrict__ r,
                                                        const CgChunk* __restrict__ chunks, CgSeg* seg, int n_seg,
                                                        double tol, double* __restrict__ partial, CgControl* ctl,
                                                        int vec_ok) {
  const CgChunk ch = chunks[blockIdx.x];
  const float alpha = seg[ch.seg].alpha;
  const bool live = seg[ch.seg].active != 0;
  float s = 0.f;
  int t0;
  cg_for_chunk(ch, vec_ok != 0, [&](long long k) {
    float4 rk = *reinterpret_cast<const float4*>(r + k);
    if (live) {
      const float4 pk = *reinterpret_cast<const float4*>(p + k);
      const float4 qk = *reinterpret_cast<const float4*>(q + k);
      float4 dk = *reinterpret_cast<const float4*>(d + k);
      dk.x = fmaf(alpha, pk.x, dk.x); dk.y = fmaf(alpha, pk.y, dk.y); dk.z = fmaf(alpha, pk.z, dk.z); dk.w = fmaf(alpha, pk.w, dk.w);
      rk.x = fmaf(-alpha, qk.x, rk.x); rk.y = fmaf(-alpha, qk.y, rk.y); rk.z = fmaf(-alpha, qk.z, rk.z); rk.w = fmaf(-alpha, qk.w, rk.w);
      *reinterpret_cast<float4*>(d + k) = dk;
      *reinterpret_cast<float4*>(r + k) = rk;
    }
    s += rk.x * rk.x + rk.y * rk.y + rk.z * rk.z + rk.w * rk.w;
  }, t0);
  for (int i = t0 + threadIdx.x; i < ch.len; i += 256) {
    const long long k = ch.start + i;
    float rk = r[k];
    if (live) {
      d[k] = fmaf(alpha, p[k], d[k]);
      rk = fmaf(-alpha, q[k], rk);
      r[k] = rk;
    }
    s = fmaf(rk, rk, s);
  }
  const double t = block_sum_256((double)s);
  if (cg_last_block(t, partial, ctl)) cg_scalars_block(2, partial, seg, n_seg, tol, ctl);
}

__global__ void __launch_bounds__(256) cg_direction_kernel(const float* __restrict__ r, float* __restrict__ p,
                                                           const CgChunk* __restrict__ chunks,
                                                           const CgSeg* __restrict__ seg, int vec_ok) {
  const CgChunk ch = chunks[blockIdx.x];
  if (seg[ch.seg].beta == 0.f && seg[ch.seg].active == 0 && seg[ch.seg].alpha == 0.f) return;  // frozen before this step
  const float beta = seg[ch.seg].beta;
  int t0;
  cg_for_chunk(ch, vec_ok != 0, [&](long long k) {
    const float4 rk = *reinterpret_cast<const float4*>(r + k);
    float4 pk = *reinterpret_cast<const float4*>(p + k);
    pk.x = fmaf(beta, pk.x, rk.x); pk.y = fmaf(beta, pk.y, rk.y); pk.z = fmaf(beta, pk.z, rk.z); pk.w = fmaf(beta, pk.w, rk.w);
    *reinterpret_cast<float4*>(p + k) = pk;
  }, t0);
  for (int i = t0 + threadIdx.x; i < ch.len; i += 256) {
    const long long k = ch.start + i;
    p[k] = fmaf(beta, p[k], r[k]);
  }
}

// ---- two-term TF32 split -----------------------------------------------------------------------
__device__ __forceinline__ float round_tf32(float x) {
  uint32_t u;
  asm("cvt.rna.tf32.f32 %0, %1;" : "=r"(u) : "f"(x));
  return __uint_as_float(u);
}

// hi = tf32(x), lo = tf32(x - hi).  x - hi is exact in FP32 (at most 13 significant bits), so the only
// loss is the rounding of lo: |x - hi - lo| <= 2^-22 |x|.
template <bool VEC>
__global__ void split_tf32_kernel(const float* __restrict__ src, int64_t rows, int cols, int64_t ld,
                                  float* __restrict__ hi, float* __restrict__ lo, int64_t ld_out) {
  const int per_row = VEC ? cols / 4 : cols;
  const int64_t total = rows * per_row;
  for (int64_t i = blockIdx.x * (int64_t)blockDim.x + threadIdx.x; i < total; i += (int64_t)gridDim.x * blockDim.x) {
    const int64_t r = i / per_row;
    const int cidx = (int)(i - r * per_row);
    if (VEC) {
      const float4 x = __ldg(reinterpret_cast<const float4*>(src + r * ld) + cidx);
      float4 h, l;
      h.x = round_tf32(x.x); l.x = round_tf32(x.x - h.x);
      h.y = round_tf32(x.y); l.y = round_tf32(x.y - h.y);
      h.z = round_tf32(x.z); l.z = round_tf32(x.z - h.z);
      h.w = round_tf32(x.w); l.w = round_tf32(x.w - h.w);
      reinterpret_cast<float4*>(hi + r * ld_out)[cidx] = h;
      reinterpret_cast<float4*>(lo + r * ld_out)[cidx] = l;
    } else {
      const float x = __ldg(src + r * ld + cidx);
      const float h = round_tf32(x);
      hi[r * ld_out + cidx] = h;
      lo[r * ld_out + cidx] = round_tf32(x - h);
    }
  }
}

}  // namespace

int launch_gather_rows(const float* src, int64_t src_rows, int cols, const int32_t* idx, int64_t n_idx,
                       float* dst, int* err_flag, cudaStream_t st) {
  if (n_idx <= 0) return 0;
  const int vec = (cols % 4 == 0) && ((reinterpret_cast<uintptr_t>(src) & 15) == 0) &&
                  ((reinterpret_cast<uintptr_t>(dst) & 15) == 0);
  const long long blocks = (n_idx + 7) / 8;
  const int grid = (int)(blocks < 148LL * 16 ? blocks : 148LL * 16);
  gather_rows_kernel<<<grid, 256, 0, st>>>(src, src_rows, cols, idx, n_idx, dst, err_flag, vec);
  return 1;
}

int64_t colsum_scratch_floats(int64_t rows, int cols) {
  return ((rows + CS_ROWS - 1) / CS_ROWS) * (int64_t)cols;
}

int launch_colsum(const float* A, int64_t rows, int cols, int64_t lda, float alpha, const float* cin,
                  float beta, float* out, float* scratch, cudaStream_t st) {
  const int parts = (int)((rows + CS_ROWS - 1) / CS_ROWS);
  const bool vec = (cols % 4 == 0) && (lda % 4 == 0) && ((reinterpret_cast<uintptr_t>(A) & 15) == 0) &&
                   ((reinterpret_cast<uintptr_t>(scratch) & 15) == 0);
  if (vec) {
    dim3 grid((cols + 127) / 128, parts);
    colsum_partial_vec_kernel<<<grid, 256, 0, st>>>(A, rows, cols, lda, scratch);
  } else {
    dim3 grid((cols + 31) / 32, parts);
    colsum_partial_kernel<<<grid, 256, 0, st>>>(A, rows, cols, lda, scratch);
  }
  colsum_final_kernel<<<(cols + 31) / 32, 256, 0, st>>>(scratch, parts, cols, alpha, cin, beta, out);
  return 2;
}

int loss_num_partials(int64_t count) { return (int)((count + LOSS_PER_BLOCK - 1) / LOSS_PER_BLOCK); }

int launch_loss_delta(const float* Z, const float* Y, int64_t count, float* delta, double* partial,
                      cudaStream_t st) {
  loss_delta_kernel<<<loss_num_partials(count), 256, 0, st>>>(Z, Y, count, delta, partial);
  return 1;
}

int launch_sum_partials(const double* partial, int count, double* out, bool accumulate, cudaStream_t st) {
  sum_partials_kernel<<<1, 256, 0, st>>>(partial, count, out, accumulate ? 1 : 0);
  return 1;
}

// Register-resident form for groups of at most 1024 * STRIPS columns (n and every group boundary multiples
// of 4): every thread keeps its n_L x 4 x STRIPS slice of D_i in registers across the passes and the streams,
// so D is read exactly once.  FLY: the factor of the last hidden layer has the closed form D_i[u][t] = W^L[u][t] *
// z (1 - z) (what factor_last_kernel stores); it is formed here, with the same two multiplications, from W^L (80 KB,
// cache-resident) and the sample's row of Z instead of being streamed from memory: 8 KB instead of 80 KB per sample
// at n_L = 10, the same bits.
template <int NLMAX, int STRIPS, bool FLY>
__global__ void __launch_bounds__(256) factor_apply_reg_kernel(const float* __restrict__ D, const float* __restrict__ U,
                                                               int nL, int n, int groups, int streams,
                                                               long long stream_stride, float* __restrict__ Q,
                                                               const float* __restrict__ WL, const float* __restrict__ Zprev) {
  __shared__ float red[8][NLMAX];
  __shared__ float pu[NLMAX];
  const long long i = blockIdx.x;
  const int col0 = (int)(((long long)blockIdx.y * n) / groups), col1 = (int)(((long long)(blockIdx.y + 1) * n) / groups);
  const float* d = D + i * nL * n;
  const int lane = threadIdx.x & 31, w = threadIdx.x >> 5;
  float4 dv[STRIPS][NLMAX];
#pragma unroll
  for (int s = 0; s < STRIPS; ++s) {
    const int j = col0 + (s * 256 + threadIdx.x) * 4;
    const bool ok = j < col1;
    if (FLY) {
      float4 ds = make_float4(0.f, 0.f, 0.f, 0.f);
      if (ok) {
        const float4 z = __ldg(reinterpret_cast<const float4*>(Zprev + i * n + j));
        ds = make_float4(z.x * (1.f - z.x), z.y * (1.f - z.y), z.z * (1.f - z.z), z.w * (1.f - z.w));
      }
#pragma unroll
      for (int u = 0; u < NLMAX; ++u) {
        float4 wv = make_float4(0.f, 0.f, 0.f, 0.f);
        if (ok && u < nL) wv = __ldg(reinterpret_cast<const float4*>(WL + (long long)u * n + j));
        dv[s][u] = make_float4(wv.x * ds.x, wv.y * ds.y, wv.z * ds.z, wv.w * ds.w);
      }
    } else {
#pragma unroll
      for (int u = 0; u < NLMAX; ++u)
        dv[s][u] = (ok && u < nL) ? __ldg(reinterpret_cast<const float4*>(d + (long long)u * n + j)) : make_float4(0.f, 0.f, 0.f, 0.f);
    }
  }
  for (int a = 0; a < streams; ++a) {
    const float* u_row = U + a * stream_stride + i * n;
    float* q_row = Q + a * stream_stride + i * n;
    float acc[NLMAX];
#pragma unroll
    for (int u = 0; u < NLMAX; ++u) acc[u] = 0.f;
#pragma unroll
    for (int s = 0; s < STRIPS; ++s) {
      const int j = col0 + (s * 256 + threadIdx.x) * 4;
      const float4 uj = j < col1 ? __ldg(reinterpret_cast<const float4*>(u_row + j)) : make_float4(0.f, 0.f, 0.f, 0.f);
#pragma unroll
      for (int u = 0; u < NLMAX; ++u)
        acc[u] += dv[s][u].x * uj.x + dv[s][u].y * uj.y + dv[s][u].z * uj.z + dv[s][u].w * uj.w;
    }
#pragma unroll
    for (int u = 0; u < NLMAX; ++u) {
      const float s = warp_sum(acc[u]);
      if (lane == 0) red[w][u] = s;
    }
    __syncthreads();
    if (threadIdx.x < NLMAX) {
      float s = 0.f;
#pragma unroll
      for (int k = 0; k < 8; ++k) s += red[k][threadIdx.x];
      pu[threadIdx.x] = 2.f * s;                              // B = 2I
    }
    __syncthreads();
#pragma unroll
    for (int s = 0; s < STRIPS; ++s) {
      const int j = col0 + (s * 256 + threadIdx.x) * 4;
      if (j < col1) {
        float4 q = make_float4(0.f, 0.f, 0.f, 0.f);
#pragma unroll
        for (int u = 0; u < NLMAX; ++u) {
          const float pv = pu[u];
          q.x = fmaf(dv[s][u].x, pv, q.x); q.y = fmaf(dv[s][u].y, pv, q.y);
          q.z = fmaf(dv[s][u].z, pv, q.z); q.w = fmaf(dv[s][u].w, pv, q.w);
        }
        *reinterpret_cast<float4*>(q_row + j) = q;
      }
    }
  }
}

int launch_factor_last(const float* WL, const float* Zprev, int64_t rows, int nL, int n, float* D, cudaStream_t st) {
  factor_last_kernel<<<(unsigned)rows, 256, 0, st>>>(WL, Zprev, nL, n, D);
  return 1;
}

int launch_factor_apply(const float* D, const float* U, int64_t rows, int nL, int n, int groups, int streams,
                        int64_t stream_stride, float* Q, cudaStream_t st) {
  bool vec = (n % 4 == 0) && (stream_stride % 4 == 0) && ((reinterpret_cast<uintptr_t>(D) & 15) == 0) &&
             ((reinterpret_cast<uintptr_t>(U) & 15) == 0) && ((reinterpret_cast<uintptr_t>(Q) & 15) == 0);
  int widest = 0;
  for (int b = 0; b < groups; ++b) {
    const int c0 = (int)(((long long)b * n) / groups), c1 = (int)(((long long)(b + 1) * n) / groups);
    if (c0 % 4 != 0) vec = false;
    if (c1 - c0 > widest) widest = c1 - c0;
  }
  const dim3 grid((unsigned)rows, (unsigned)groups);
  const long long ss = stream_stride;
#define GN_FA_REG(NL, STR) { factor_apply_reg_kernel<NL, STR, false><<<grid, 256, 0, st>>>(D, U, nL, n, groups, streams, ss, Q, nullptr, nullptr); return 1; }
  if (vec && widest <= 1024 && nL <= 4)  GN_FA_REG(4, 1)
  if (vec && widest <= 1024 && nL <= 10) GN_FA_REG(10, 1)
  if (vec && widest <= 2048 && nL <= 4)  GN_FA_REG(4, 2)
  if (vec && widest <= 2048 && nL <= 10) GN_FA_REG(10, 2)
  if (vec && widest <= 1024 && nL <= 16) GN_FA_REG(16, 1)
#undef GN_FA_REG
  if (nL <= 4) factor_apply_kernel<4><<<grid, 256, 0, st>>>(D, U, nL, n, groups, streams, ss, Q);
  else if (nL <= 10) factor_apply_kernel<10><<<grid, 256, 0, st>>>(D, U, nL, n, groups, streams, ss, Q);
  else if (nL <= 16) factor_apply_kernel<16><<<grid, 256, 0, st>>>(D, U, nL, n, groups, streams, ss, Q);
  else factor_apply_kernel<32><<<grid, 256, 0, st>>>(D, U, nL, n, groups, streams, ss, Q);
  return 1;
}

// The same product for the last hidden layer without its stored factor (see factor_apply_reg_kernel): one group, one
// stream.  Returns 0, having launched nothing, if the register-resident form does not take the shape.
int launch_factor_apply_last(const float* WL, const float* Zprev, const float* U, int64_t rows, int nL, int n, float* Q,
                             cudaStream_t st) {
  const bool vec = (n % 4 == 0) && ((reinterpret_cast<uintptr_t>(WL) & 15) == 0) && ((reinterpret_cast<uintptr_t>(Zprev) & 15) == 0) &&
                   ((reinterpret_cast<uintptr_t>(U) & 15) == 0) && ((reinterpret_cast<uintptr_t>(Q) & 15) == 0);
  if (!vec) return 0;
  const dim3 grid((unsigned)rows, 1);
#define GN_FA_FLY(NL, STR) { factor_apply_reg_kernel<NL, STR, true><<<grid, 256, 0, st>>>(nullptr, U, nL, n, 1, 1, 0, Q, WL, Zprev); return 1; }
  if (n <= 1024 && nL <= 4)  GN_FA_FLY(4, 1)
  if (n <= 1024 && nL <= 10) GN_FA_FLY(10, 1)
  if (n <= 2048 && nL <= 4)  GN_FA_FLY(4, 2)
  if (n <= 2048 && nL <= 10) GN_FA_FLY(10, 2)
  if (n <= 1024 && nL <= 16) GN_FA_FLY(16, 1)
#undef GN_FA_FLY
  return 0;
}

int launch_axpby(int64_t n, float a, const float* x, float b, const float* y, float* out, cudaStream_t st) {
  long long blocks = (n + 255) / 256;
  if (blocks > 148LL * 16) blocks = 148LL * 16;
  axpby_kernel<<<(unsigned)blocks, 256, 0, st>>>(n, a, x, b, y, out);
  return 1;
}

int launch_split_tf32(const float* src, int64_t rows, int cols, int64_t ld, float* hi, float* lo, int64_t ld_out,
                      cudaStream_t st) {
  if (rows < 1 || cols < 1) return 0;
  const bool vec = cols % 4 == 0 && ld % 4 == 0 && ld_out % 4 == 0 && (reinterpret_cast<uintptr_t>(src) & 15) == 0 &&
                   (reinterpret_cast<uintptr_t>(hi) & 15) == 0 && (reinterpret_cast<uintptr_t>(lo) & 15) == 0;
  const int64_t total = rows * (vec ? cols / 4 : cols);
  int64_t blocks = (total + 255) / 256;
  if (blocks > 148 * 16) blocks = 148 * 16;
  if (vec) split_tf32_kernel<true><<<(int)blocks, 256, 0, st>>>(src, rows, cols, ld, hi, lo, ld_out);
  else     split_tf32_kernel<false><<<(int)blocks, 256, 0, st>>>(src, rows, cols, ld, hi, lo, ld_out);
  return 1;
}

namespace {
inline int all_aligned16(std::initializer_list<const void*> ps) {
  for (const void* q : ps)
    if (reinterpret_cast<uintptr_t>(q) & 15) return 0;
  return 1;
}
}  // namespace

int launch_cg_init(const float* g, float* d, float* r, float* p, const CgChunk* chunks, int n_chunks,
                   double* partial, CgSeg* seg, int n_seg, double tol, CgControl* ctl, cudaStream_t st) {
  cg_init_kernel<<<n_chunks, 256, 0, st>>>(g, d, r, p, chunks, partial, seg, n_seg, tol, ctl, all_aligned16({g, d, r, p}));
  return 1;
}
int launch_cg_dot(const float* p, const float* q, const CgChunk* chunks, int n_chunks, double* partial,
                  CgSeg* seg, int n_seg, CgControl* ctl, cudaStream_t st) {
  cg_dot_kernel<<<n_chunks, 256, 0, st>>>(p, q, chunks, partial, seg, n_seg, ctl, all_aligned16({p, q}));
  return 1;
}
int launch_cg_update(const float* p, const float* q, float* d, float* r, const CgChunk* chunks,
                     int n_chunks, CgSeg* seg, int n_seg, double tol, double* partial, CgControl* ctl, cudaStream_t st) {
  cg_update_kernel<<<n_chunks, 256, 0, st>>>(p, q, d, r, chunks, seg, n_seg, tol, partial, ctl, all_aligned16({p, q, d, r}));
  return 1;
}
int launch_cg_direction(const float* r, float* p, const CgChunk* chunks, int n_chunks, const CgSeg* seg,
                        cudaStream_t st) {
  cg_direction_kernel<<<n_chunks, 256, 0, st>>>(r, p, chunks, seg, all_aligned16({r, p}));
  return 1;
}

}  // namespace gn
