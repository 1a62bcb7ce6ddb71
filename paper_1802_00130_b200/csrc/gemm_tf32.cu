// TF32 tensor-core GEMM for sm_100a: tcgen05.mma with the accumulator in tensor memory, operands
// staged in shared memory by TMA (128-byte swizzle), fused epilogue read back with tcgen05.ld.
//
// One CTA computes one 128 x BN output tile.  Warp roles:
//   warp 0      TMA producer (one elected lane): fills a ring of STAGES operand buffers
//   warp 1      MMA issuer   (one elected lane): 4 x (128 x BN x 8) tcgen05.mma per ring slot
//   warps 2..5  epilogue: each owns one 32-lane quadrant of tensor memory
// Up to two (A, B) operand pairs are accumulated into the same tile (the forward directional
// derivative needs R z^{m-1} W^m + z^{m-1} V^m in one accumulator).
//
// Operand layouts in shared memory (32-bit elements, rows of 128 B):
//   K-major  : rows = M (or N) index, 32 consecutive K elements per row; plain 128-byte swizzle
//              (16-byte units permuted over 8 rows).  Descriptor: stride between 8-row groups
//              1024 B; one MMA (K = 8) advances 32 B inside the row.
//   MN-major : the global operand is [K][MN] with MN contiguous; it is staged as chunks of 32 MN
//              elements, each chunk = BK rows (K index) of 128 B.  32-bit MN-major operands must
//              use the 128-byte swizzle with 32-byte atoms (32-byte units permuted over 4 rows), in
//              the tensor map and in the descriptor alike.  Descriptor: leading-dimension offset =
//              chunk size (BK * 128 B), stride between 4-row groups 512 B; one MMA (K = 8)
//              advances 1024 B.
// Every wait on an mbarrier is bounded: after about two seconds the waiting role records an error
// code in global memory and the CTA drains and exits (tensor memory is always released).
#include <cuda.h>

#include "gn_kernels.h"

namespace gn {
namespace {

constexpr int BM = 128, BK = 32;
constexpr int A_STAGE_BYTES = BM * BK * 4;  // 16 KB
constexpr unsigned long long WAIT_LIMIT_NS = 2000000000ull;

struct Tf32Params {
  int M, N;
  int kblocks[2];
  int a_mn, b_mn;
  float* D; long long ldd;
  const float* bias; int sigmoid;
  const float* dsig; long long ld_dsig; int dsig_rows;
  float alpha;
  const float* cin; long long ld_cin; float beta;
  int vec_epi;
  int tiles_n;
  int* err;
};

__device__ __forceinline__ uint32_t smem_u32(const void* p) { return (uint32_t)__cvta_generic_to_shared(p); }

__device__ __forceinline__ unsigned long long globaltimer() {
  unsigned long long t;
  asm volatile("mov.u64 %0, %globaltimer;" : "=l"(t));
  return t;
}

__device__ __forceinline__ void mbar_init(uint64_t* bar, uint32_t count) {
  asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(smem_u32(bar)), "r"(count));
}
__device__ __forceinline__ void mbar_expect_tx(uint64_t* bar, uint32_t bytes) {
  asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(smem_u32(bar)), "r"(bytes) : "memory");
}
__device__ __forceinline__ bool mbar_try_wait(uint64_t* bar, uint32_t parity) {
  uint32_t ok;
  asm volatile(
      "{\n\t.reg .pred p;\n\t"
      "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\t"
      "selp.u32 %0, 1, 0, p;\n\t}"
      : "=r"(ok) : "r"(smem_u32(bar)), "r"(parity) : "memory");
  return ok != 0;
}
// Bounded wait.  Returns false (and records `code`) if the phase did not complete in time.
__device__ __forceinline__ bool mbar_wait(uint64_t* bar, uint32_t parity, int* err, int code) {
  if (mbar_try_wait(bar, parity)) return true;
  const unsigned long long t0 = globaltimer();
  while (!mbar_try_wait(bar, parity)) {
    if (globaltimer() - t0 > WAIT_LIMIT_NS) {
      atomicCAS(err, 0, code);
      return false;
    }
  }
  return true;
}

__device__ __forceinline__ void tma_load_2d(void* dst, const CUtensorMap* map, int x, int y, uint64_t* bar) {
  asm volatile(
      "cp.async.bulk.tensor.2d.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%2, %3}], [%4];"
      ::"r"(smem_u32(dst)), "l"(reinterpret_cast<uint64_t>(map)), "r"(x), "r"(y), "r"(smem_u32(bar))
      : "memory");
}

// layout: 2 = 128-byte swizzle (16-byte atoms), 1 = 128-byte swizzle with 32-byte atoms
__device__ __forceinline__ uint64_t make_desc(uint32_t saddr, uint32_t lbo_bytes, uint32_t sbo_bytes, uint32_t layout) {
  uint64_t d = 0;
  d |= (uint64_t)((saddr >> 4) & 0x3FFF);
  d |= (uint64_t)((lbo_bytes >> 4) & 0x3FFF) << 16;
  d |= (uint64_t)((sbo_bytes >> 4) & 0x3FFF) << 32;
  d |= (uint64_t)1 << 46;  // descriptor version of this architecture
  d |= (uint64_t)layout << 61;
  return d;
}

__device__ __forceinline__ void mma_tf32(uint32_t tmem_d, uint64_t adesc, uint64_t bdesc, uint32_t idesc, uint32_t accum) {
  asm volatile(
      "{\n\t.reg .pred p;\n\t"
      "setp.ne.b32 p, %4, 0;\n\t"
      "tcgen05.mma.cta_group::1.kind::tf32 [%0], %1, %2, %3, p;\n\t}"
      ::"r"(tmem_d), "l"(adesc), "l"(bdesc), "r"(idesc), "r"(accum) : "memory");
}
__device__ __forceinline__ void mma_commit(uint64_t* bar) {
  asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(smem_u32(bar)) : "memory");
}
__device__ __forceinline__ void tc_fence_after() { asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void tc_fence_before() { asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory"); }

__device__ __forceinline__ void tmem_ld32(uint32_t taddr, float (&v)[32]) {
  uint32_t r[32];
  asm volatile(
      "tcgen05.ld.sync.aligned.32x32b.x32.b32 "
      "{%0, %1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15, "
      "%16, %17, %18, %19, %20, %21, %22, %23, %24, %25, %26, %27, %28, %29, %30, %31}, [%32];"
      : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7]),
        "=r"(r[8]), "=r"(r[9]), "=r"(r[10]), "=r"(r[11]), "=r"(r[12]), "=r"(r[13]), "=r"(r[14]), "=r"(r[15]),
        "=r"(r[16]), "=r"(r[17]), "=r"(r[18]), "=r"(r[19]), "=r"(r[20]), "=r"(r[21]), "=r"(r[22]), "=r"(r[23]),
        "=r"(r[24]), "=r"(r[25]), "=r"(r[26]), "=r"(r[27]), "=r"(r[28]), "=r"(r[29]), "=r"(r[30]), "=r"(r[31])
      : "r"(taddr));
  asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory");
#pragma unroll
  for (int i = 0; i < 32; ++i) v[i] = __uint_as_float(r[i]);
}

template <int BN, int STAGES>
__global__ void __launch_bounds__(192, 1)
gemm_tf32_kernel(const __grid_constant__ CUtensorMap tmA0, const __grid_constant__ CUtensorMap tmB0,
                 const __grid_constant__ CUtensorMap tmA1, const __grid_constant__ CUtensorMap tmB1,
                 const Tf32Params p) {
  constexpr int B_STAGE_BYTES = BN * BK * 4;
  constexpr int STAGE_BYTES = A_STAGE_BYTES + B_STAGE_BYTES;
  extern __shared__ uint8_t smem_raw[];
  uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~(uintptr_t)1023);
  uint64_t* full = reinterpret_cast<uint64_t*>(smem + STAGES * STAGE_BYTES);
  uint64_t* empty = full + STAGES;
  uint64_t* tmem_full = empty + STAGES;
  uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(tmem_full + 1);

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int tile_m = blockIdx.x / p.tiles_n, tile_n = blockIdx.x % p.tiles_n;
  const int m0 = tile_m * BM, n0 = tile_n * BN;
  const int total_kb = p.kblocks[0] + p.kblocks[1];

  if (threadIdx.x == 0) {
    for (int s = 0; s < STAGES; ++s) { mbar_init(&full[s], 1); mbar_init(&empty[s], 1); }
    mbar_init(tmem_full, 1);
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  if (warp == 2) {  // tensor-memory allocation: BN columns of 128 lanes x 32 bit
    asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(tmem_slot)), "r"(BN) : "memory");
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
  }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem_base = *tmem_slot;

  if (warp == 0) {
    if (lane == 0) {
      // ---------------------------------------------------------------- producer
      for (int kb = 0; kb < total_kb; ++kb) {
        const int s = kb % STAGES;
        const uint32_t ph = (kb / STAGES) & 1;
        if (!mbar_wait(&empty[s], ph ^ 1, p.err, 1)) break;
        const int pair = kb < p.kblocks[0] ? 0 : 1;
        const int k0 = (pair == 0 ? kb : kb - p.kblocks[0]) * BK;
        const CUtensorMap* ma = pair == 0 ? &tmA0 : &tmA1;
        const CUtensorMap* mb = pair == 0 ? &tmB0 : &tmB1;
        uint8_t* sa = smem + s * STAGE_BYTES;
        uint8_t* sb = sa + A_STAGE_BYTES;
        mbar_expect_tx(&full[s], STAGE_BYTES);
        if (!p.a_mn) {
          tma_load_2d(sa, ma, k0, m0, &full[s]);
        } else {
#pragma unroll
          for (int c = 0; c < BM / 32; ++c) tma_load_2d(sa + c * (BK * 128), ma, m0 + 32 * c, k0, &full[s]);
        }
        if (!p.b_mn) {
          tma_load_2d(sb, mb, k0, n0, &full[s]);
        } else {
#pragma unroll
          for (int c = 0; c < BN / 32; ++c) tma_load_2d(sb + c * (BK * 128), mb, n0 + 32 * c, k0, &full[s]);
        }
      }
    }
  } else if (warp == 1) {
    if (lane == 0) {
      // ---------------------------------------------------------------- MMA issuer
      // instruction descriptor: D = F32, A = B = TF32, majors, N >> 3, M >> 4
      const uint32_t idesc = (1u << 4) | (2u << 7) | (2u << 10) | ((uint32_t)(p.a_mn ? 1 : 0) << 15) |
                             ((uint32_t)(p.b_mn ? 1 : 0) << 16) | ((uint32_t)(BN >> 3) << 17) | ((uint32_t)(BM >> 4) << 24);
      const uint32_t a_lbo = p.a_mn ? BK * 128 : 16, b_lbo = p.b_mn ? BK * 128 : 16;
      const uint32_t a_step = p.a_mn ? 1024 : 32, b_step = p.b_mn ? 1024 : 32;
      const uint32_t a_sbo = p.a_mn ? 512 : 1024, b_sbo = p.b_mn ? 512 : 1024;
      const uint32_t a_lay = p.a_mn ? 1 : 2, b_lay = p.b_mn ? 1 : 2;
      bool ok = true;
      for (int kb = 0; kb < total_kb && ok; ++kb) {
        const int s = kb % STAGES;
        const uint32_t ph = (kb / STAGES) & 1;
        ok = mbar_wait(&full[s], ph, p.err, 2);
        if (!ok) break;
        tc_fence_after();
        const uint32_t sa = smem_u32(smem + s * STAGE_BYTES);
        const uint32_t sb = sa + A_STAGE_BYTES;
#pragma unroll
        for (int k = 0; k < BK / 8; ++k) {
          const uint64_t ad = make_desc(sa + k * a_step, a_lbo, a_sbo, a_lay);
          const uint64_t bd = make_desc(sb + k * b_step, b_lbo, b_sbo, b_lay);
          mma_tf32(tmem_base, ad, bd, idesc, (kb | k) != 0 ? 1u : 0u);
        }
        mma_commit(&empty[s]);  // frees the slot once these MMAs have read it
      }
      mma_commit(tmem_full);    // accumulator complete (also reached after a timed-out wait)
    }
  } else {
    // ------------------------------------------------------------------ epilogue (warps 2..5)
    const int quad = warp & 3;  // tensor-memory lanes 32*quad .. 32*quad+31 are this warp's
    const bool ready = mbar_wait(tmem_full, 0, p.err, 3);
    tc_fence_after();
    const int m = m0 + quad * 32 + lane;
    if (ready) {
      const long long zrow = p.dsig ? (long long)(m % p.dsig_rows) * p.ld_dsig : 0;
      for (int c = 0; c < BN / 32; ++c) {
        const int nb = n0 + c * 32;
        if (nb >= p.N) break;               // warp-uniform
        float v[32];
        tmem_ld32(tmem_base + ((uint32_t)(quad * 32) << 16) + (uint32_t)(c * 32), v);
        if (m >= p.M) continue;
#pragma unroll
        for (int q = 0; q < 8; ++q) {
          const int n = nb + q * 4;
          if (n >= p.N) break;
          const int cnt = min(4, p.N - n);
          const bool v4 = p.vec_epi && cnt == 4;
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
          float t[4];
#pragma unroll
          for (int j = 0; j < 4; ++j) {
            float x = v[q * 4 + j] + bz[j];
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
    tc_fence_before();
  }
  __syncthreads();
  if (warp == 2) {
    tc_fence_after();
    asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem_base), "r"(BN) : "memory");
  }
}

// ---- host side ---------------------------------------------------------------------------------
typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*,
                                  const cuuint64_t*, const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave,
                                  CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

EncodeTiledFn encode_fn() {
  static EncodeTiledFn fn = nullptr;
  static bool tried = false;
  if (!tried) {
    tried = true;
    void* p = nullptr;
    cudaDriverEntryPointQueryResult q;
    if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &p, cudaEnableDefault, &q) == cudaSuccess &&
        q == cudaDriverEntryPointSuccess)
      fn = reinterpret_cast<EncodeTiledFn>(p);
    else
      cudaGetLastError();
  }
  return fn;
}

// 2-D map over a row-major [rows][cols] float matrix with leading dimension ld; box = (box_c, box_r).
bool make_map(CUtensorMap* m, const float* base, long long rows, long long cols, long long ld, int box_c, int box_r,
              CUtensorMapSwizzle swz) {
  EncodeTiledFn fn = encode_fn();
  if (!fn) return false;
  cuuint64_t dims[2] = {(cuuint64_t)cols, (cuuint64_t)rows};
  cuuint64_t strides[1] = {(cuuint64_t)ld * 4};
  cuuint32_t box[2] = {(cuuint32_t)box_c, (cuuint32_t)box_r};
  cuuint32_t estr[2] = {1, 1};
  CUresult r = fn(m, CU_TENSOR_MAP_DATA_TYPE_TFLOAT32, 2, const_cast<float*>(base), dims, strides, box, estr,
                  CU_TENSOR_MAP_INTERLEAVE_NONE, swz, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                  CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
  return r == CUDA_SUCCESS;
}

inline bool aligned16(const void* p) { return (reinterpret_cast<uintptr_t>(p) & 15) == 0; }

constexpr int kBN = 256, kStages = 4;
constexpr int kSmemBytes = kStages * (A_STAGE_BYTES + kBN * BK * 4) + 1024 + 256;

}  // namespace

bool gemm_tf32_eligible(const GemmArgs& g) {
  if (g.M < 1 || g.N < 32) return false;
  if (!aligned16(g.A1) || !aligned16(g.B1) || g.lda1 % 4 || g.ldb1 % 4) return false;
  if (g.A2 && (!aligned16(g.A2) || !aligned16(g.B2) || g.lda2 % 4 || g.ldb2 % 4)) return false;
  if (!encode_fn()) return false;
  return true;
}

int launch_gemm_tf32(const GemmArgs& g, int* err_flag, cudaStream_t st) {
  static bool attr_set = false;
  if (!attr_set) {
    cudaFuncSetAttribute(gemm_tf32_kernel<kBN, kStages>, cudaFuncAttributeMaxDynamicSharedMemorySize, kSmemBytes);
    attr_set = true;
  }
  CUtensorMap maps[4];
  const float* As[2] = {g.A1, g.A2};
  const float* Bs[2] = {g.B1, g.B2};
  const int Ks[2] = {g.K1, g.A2 ? g.K2 : 0};
  const long long lda[2] = {g.lda1, g.lda2}, ldb[2] = {g.ldb1, g.ldb2};
  for (int s = 0; s < 2; ++s) {
    const int src = As[s] ? s : 0;  // unused second pair: repeat the first (never dereferenced)
    bool ok;
    const CUtensorMapSwizzle kmaj = CU_TENSOR_MAP_SWIZZLE_128B, mnmaj = CU_TENSOR_MAP_SWIZZLE_128B_ATOM_32B;
    if (g.a_kmajor) ok = make_map(&maps[2 * s], As[src], g.M, Ks[src], lda[src], BK, BM, kmaj);
    else            ok = make_map(&maps[2 * s], As[src], Ks[src], g.M, lda[src], 32, BK, mnmaj);
    if (g.b_kmajor) ok = ok && make_map(&maps[2 * s + 1], Bs[src], g.N, Ks[src], ldb[src], BK, kBN, kmaj);
    else            ok = ok && make_map(&maps[2 * s + 1], Bs[src], Ks[src], g.N, ldb[src], 32, BK, mnmaj);
    if (!ok) return -1;
  }
  Tf32Params p{};
  p.M = g.M; p.N = g.N;
  p.kblocks[0] = (Ks[0] + BK - 1) / BK;
  p.kblocks[1] = (Ks[1] + BK - 1) / BK;
  p.a_mn = g.a_kmajor ? 0 : 1; p.b_mn = g.b_kmajor ? 0 : 1;
  p.D = g.D; p.ldd = g.ldd;
  p.bias = g.bias; p.sigmoid = g.sigmoid;
  p.dsig = g.dsig; p.ld_dsig = g.ld_dsig; p.dsig_rows = g.dsig_rows > 0 ? g.dsig_rows : 1;
  p.alpha = g.alpha;
  p.cin = g.cin; p.ld_cin = g.ld_cin; p.beta = g.beta;
  p.vec_epi = aligned16(g.D) && (g.ldd % 4 == 0) && (!g.bias || aligned16(g.bias)) &&
              (!g.dsig || (aligned16(g.dsig) && g.ld_dsig % 4 == 0)) &&
              (!g.cin || (aligned16(g.cin) && g.ld_cin % 4 == 0));
  p.tiles_n = (g.N + kBN - 1) / kBN;
  p.err = err_flag;
  const long long tiles = (long long)((g.M + BM - 1) / BM) * p.tiles_n;
  gemm_tf32_kernel<kBN, kStages><<<(unsigned)tiles, 192, kSmemBytes, st>>>(maps[0], maps[1], maps[2], maps[3], p);
  return 1;
}

}  // namespace gn
