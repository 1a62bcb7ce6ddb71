// TF32 tensor-core GEMM for sm_100a: tcgen05.mma with the accumulator in tensor memory, operands
// staged in shared memory by TMA (128-byte swizzle), fused epilogue read back with tcgen05.ld.
//
// Persistent kernel, one CTA per SM, each walking 128 x bn output tiles.  Warp roles:
//   warp 0      TMA producer: fills a ring of STAGES operand buffers (issue spread over lanes)
//   warp 1      MMA issuer   (one elected lane): 4 x (128 x bn x 8) tcgen05.mma per ring slot
//   warps 2..9  epilogue: two warps per 32-lane quadrant of tensor memory, alternating over the
//               tile's 32-column chunks; registers only (shared-memory bandwidth belongs to the
//               MMA and TMA), all of a chunk's global reads issued before the accumulator is read
// Two accumulators alternate in tensor memory, so a tile's epilogue overlaps the next tile's MMAs.
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

#include <utility>

#include "gn_kernels.h"

namespace gn {
namespace {

constexpr int BM = 128, BK = 32, BN_MAX = 256;
constexpr int A_STAGE_BYTES = BM * BK * 4;  // 16 KB
constexpr unsigned long long WAIT_LIMIT_NS = 2000000000ull;

struct Tf32Params {
  int M, N;
  int kblocks[2];
  int a_mn, b_mn;
  int a_3d, b_3d;       // MN-major operand fetched with one 3-D box per stage (needs a padded operand)
  float* D; long long ldd;
  const float* bias; int sigmoid;
  const float* dsig; long long ld_dsig; int dsig_rows, dsig_div;
  float alpha;
  const float* cin; long long ld_cin; float beta;
  int vec_epi;          // D, bias, dsig, cin all 16-byte aligned with leading dimensions % 4 == 0
  // error-compensated kernel only: also write the two-term TF32 split of every stored value (hi = value rounded to
  // TF32, lo = value - hi rounded to TF32) to these matrices, for the contraction that takes D as an operand next
  float* Dhi; float* Dlo; long long ld_parts;
  int bn;               // tile width: multiple of 32, 32 <= bn <= 256
  int tiles_n, tiles;
  int* err;
  // work list of the two-CTA kernel: pair q runs tiles q, q + P, ... for `waves` full waves of P tiles;
  // the `rem` tiles left over are each cut along K into `slices` parts, one per pair, done before the
  // pair's whole tiles (slices == 1: whole tiles, done last)
  int P, waves, rem, slices;
  float* sk_ws;          // [P][2][128][256] raw partial accumulators of the sliced tiles, slot = pair
  int* sk_flags;         // [P] arrival counters, one per sliced tile; zero between launches (the kernel resets them)
};

// Up to MAX_GROUP independent problems in one launch of the two-CTA kernel.  Pair q runs, problem after problem,
// its tiles of the problem's whole waves (q, q + P, ...) and then tiles rstart[g][q] .. rstart[g][q + 1] - 1 of the
// tiles left over after those waves; the host deals the left-over tiles so that the pairs' total loads come out even
// (longest tiles first), which lets the short tiles of one problem fill the partial last wave of another.
constexpr int MAX_GROUP = 6;
constexpr int MAX_PAIRS_LAUNCH = 80;        // >= SMs / 2
struct GroupParams {
  int n_prob;
  Tf32Params pr[MAX_GROUP];
  unsigned short rstart[MAX_GROUP][MAX_PAIRS_LAUNCH + 1];
  // Dependent problems in one launch (a chain of layers): problem g may read, as an operand, what problem
  // dep_prob[g] (earlier in the list) writes.  dep_all[g] == 0: a tile of g needs the producer's tiles of the
  // same 256-row panel (its A rows are the producer's output rows); dep_all[g] == 1: it needs all of them (its
  // K runs over the producer's rows).  The epilogue warps of a producer count finished tiles per panel
  // (signal bit 0) and in total (bit 1) in `done`; the TMA warps of a consumer wait, bounded, for the count.
  // Every pair works through the problems in list order and all pairs are resident, so a wait is always for
  // work that is running or about to run on another pair.
  int dep_prob[MAX_GROUP];
  int dep_all[MAX_GROUP];
  int signal[MAX_GROUP];
  int* done;                 // [n_prob][done_stride]: entry i < done_stride - 1 counts panel i, the last entry all tiles
  int done_stride;
};
struct GroupMaps { CUtensorMap m[MAX_GROUP][4]; };   // per problem: A0, B0, A1, B1

__device__ __forceinline__ uint32_t smem_u32(const void* p) { return (uint32_t)__cvta_generic_to_shared(p); }

__device__ __forceinline__ unsigned long long globaltimer() {
  unsigned long long t;
  asm volatile("mov.u64 %0, %globaltimer;" : "=l"(t));
  return t;
}

// Programmatic dependent launch.  The kernels below are launched with the stream-serialisation attribute, so
// their CTAs may become resident, set up their barriers and allocate tensor memory while the kernel before
// them in the stream is still draining; nothing of global memory is touched before grid_dep_wait() returns,
// which is when that kernel has completed and its writes are visible.  grid_dep_launch() lets the kernel
// after this one do the same.  Without the attribute both are no-ops.
__device__ __forceinline__ void grid_dep_wait() { asm volatile("griddepcontrol.wait;" ::: "memory"); }
__device__ __forceinline__ void grid_dep_launch() { asm volatile("griddepcontrol.launch_dependents;" ::: "memory"); }

__device__ __forceinline__ float round_tf32(float x) {
  uint32_t u;
  asm("cvt.rna.tf32.f32 %0, %1;" : "=r"(u) : "f"(x));
  return __uint_as_float(u);
}

__device__ __forceinline__ void mbar_init(uint64_t* bar, uint32_t count) {
  asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(smem_u32(bar)), "r"(count));
}
__device__ __forceinline__ void mbar_expect_tx(uint64_t* bar, uint32_t bytes) {
  asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(smem_u32(bar)), "r"(bytes) : "memory");
}
__device__ __forceinline__ bool mbar_test_wait(uint64_t* bar, uint32_t parity) {
  uint32_t ok;
  asm volatile(
      "{\n\t.reg .pred p;\n\t"
      "mbarrier.test_wait.parity.shared::cta.b64 p, [%1], %2;\n\t"
      "selp.u32 %0, 1, 0, p;\n\t}"
      : "=r"(ok) : "r"(smem_u32(bar)), "r"(parity) : "memory");
  return ok != 0;
}

// Potentially blocking form: the thread may be suspended until the phase completes or about `ns` nanoseconds
// have passed, instead of re-issuing the test in a loop (a spinning warp takes issue slots and load/store-unit
// queue entries from the working warps of its scheduler).
__device__ __forceinline__ bool mbar_try_wait(uint64_t* bar, uint32_t parity, uint32_t ns) {
  uint32_t ok;
  asm volatile(
      "{\n\t.reg .pred p;\n\t"
      "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2, %3;\n\t"
      "selp.u32 %0, 1, 0, p;\n\t}"
      : "=r"(ok) : "r"(smem_u32(bar)), "r"(parity), "r"(ns) : "memory");
  return ok != 0;
}

__device__ __forceinline__ void tma_load_2d(void* dst, const CUtensorMap* map, int x, int y, uint64_t* bar) {
  asm volatile(
      "cp.async.bulk.tensor.2d.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%2, %3}], [%4];"
      ::"r"(smem_u32(dst)), "l"(reinterpret_cast<uint64_t>(map)), "r"(x), "r"(y), "r"(smem_u32(bar))
      : "memory");
}

__device__ __forceinline__ void tma_load_3d(void* dst, const CUtensorMap* map, int x, int y, int z, uint64_t* bar) {
  asm volatile(
      "cp.async.bulk.tensor.3d.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%2, %3, %4}], [%5];"
      ::"r"(smem_u32(dst)), "l"(reinterpret_cast<uint64_t>(map)), "r"(x), "r"(y), "r"(z), "r"(smem_u32(bar))
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

// Accumulator read in the 16 x 256-bit fragment shape: one instruction covers 16 tensor-memory lanes (rows) and
// 32 columns; thread t of the warp receives, in register 4j + 2e + i (j = 0..3, e = 0..1, i = 0..1), the element
// of row (t / 4) + 8 e and column 8 j + 2 (t mod 4) + i.  Four neighbouring threads hold 32 contiguous bytes of a
// row, so a warp-wide 8-byte access to global memory touches 8 rows x one full 32-byte sector each, where the
// 32 x 32-bit shape (lane = row) makes every access touch 32 rows x half a sector: half the requests per byte
// on the load/store unit, which is what the epilogue is bound by.  The caller waits (tmem_ld_wait) before use.
__device__ __forceinline__ void tmem_ld_16x256b_x4(uint32_t taddr, float* v) {
  uint32_t r[16];
  asm volatile(
      "tcgen05.ld.sync.aligned.16x256b.x4.b32 "
      "{%0, %1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15}, [%16];"
      : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7]),
        "=r"(r[8]), "=r"(r[9]), "=r"(r[10]), "=r"(r[11]), "=r"(r[12]), "=r"(r[13]), "=r"(r[14]), "=r"(r[15])
      : "r"(taddr));
#pragma unroll
  for (int i = 0; i < 16; ++i) v[i] = __uint_as_float(r[i]);
}
__device__ __forceinline__ void tmem_ld_wait() { asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory"); }

__device__ __forceinline__ int ld_acquire_gpu(const int* p) {
  int v;
  asm volatile("ld.acquire.gpu.global.s32 %0, [%1];" : "=r"(v) : "l"(p) : "memory");
  return v;
}

__device__ __forceinline__ void mbar_arrive(uint64_t* bar) {
  asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(smem_u32(bar)) : "memory");
}

// Bounded wait that also gives up at once when another role of this CTA has already failed.
__device__ __forceinline__ bool wait_or_abort(uint64_t* bar, uint32_t parity, volatile int* abort_flag, int* err, int code) {
  if (mbar_test_wait(bar, parity)) return true;
  const unsigned long long t0 = globaltimer();
  while (!mbar_try_wait(bar, parity, 100000u)) {     // wakes at the latest every ~0.1 ms to look at the clock
    if (*abort_flag) return false;
    if (globaltimer() - t0 > WAIT_LIMIT_NS) {
      atomicCAS(err, 0, code);
      *abort_flag = 1;
      return false;
    }
  }
  return true;
}

// Persistent kernel: CTA b works on tiles b, b + gridDim.x, ...  Tile = 128 rows x p.bn columns
// (p.bn a multiple of 32, at most 256).  Two accumulators of 256 tensor-memory columns alternate so
// that the epilogue of one tile overlaps the MMAs of the next.
template <int STAGES>
__global__ void __launch_bounds__(320, 1)
gemm_tf32_kernel(const __grid_constant__ CUtensorMap tmA0, const __grid_constant__ CUtensorMap tmB0,
                 const __grid_constant__ CUtensorMap tmA1, const __grid_constant__ CUtensorMap tmB1,
                 const Tf32Params p) {
  constexpr int B_STAGE_MAX = BN_MAX * BK * 4;
  constexpr int STAGE_BYTES = A_STAGE_BYTES + B_STAGE_MAX;
  extern __shared__ uint8_t smem_raw[];
  uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~(uintptr_t)1023);
  uint64_t* full = reinterpret_cast<uint64_t*>(smem + STAGES * STAGE_BYTES);
  uint64_t* empty = full + STAGES;
  uint64_t* acc_full = empty + STAGES;   // [2]
  uint64_t* acc_empty = acc_full + 2;    // [2]
  uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(acc_empty + 2);
  volatile int* abort_flag = reinterpret_cast<volatile int*>(tmem_slot + 1);

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int total_kb = p.kblocks[0] + p.kblocks[1];
  const int bn = p.bn;
  const uint32_t stage_tx = A_STAGE_BYTES + (uint32_t)bn * BK * 4;

  if (threadIdx.x == 0) {
    for (int s = 0; s < STAGES; ++s) { mbar_init(&full[s], 1); mbar_init(&empty[s], 1); }
    for (int b = 0; b < 2; ++b) { mbar_init(&acc_full[b], 1); mbar_init(&acc_empty[b], 8); }
    *abort_flag = 0;
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  if (warp == 2) {  // all 512 tensor-memory columns: two 128 x 256 FP32 accumulators
    asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(tmem_slot)), "r"(512) : "memory");
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
  }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem_base = *tmem_slot;
  grid_dep_wait();
  grid_dep_launch();

  if (warp == 0) {
    // ------------------------------------------------------------------ producer (TMA issue spread over lanes)
    int it = 0;
    bool ok = true;
    for (int t = blockIdx.x; t < p.tiles && ok; t += gridDim.x) {
      const int m0 = (t / p.tiles_n) * BM, n0 = (t % p.tiles_n) * bn;
      for (int kb = 0; kb < total_kb; ++kb, ++it) {
        const int s = it % STAGES;
        const uint32_t ph = (it / STAGES) & 1;
        int good = 1;
        if (lane == 0) good = wait_or_abort(&empty[s], ph ^ 1, abort_flag, p.err, 1) ? 1 : 0;
        good = __shfl_sync(0xffffffffu, good, 0);
        if (!good) { ok = false; break; }
        if (lane == 0) mbar_expect_tx(&full[s], stage_tx);
        __syncwarp();
        const int pair = kb < p.kblocks[0] ? 0 : 1;
        const int k0 = (pair == 0 ? kb : kb - p.kblocks[0]) * BK;
        const CUtensorMap* ma = pair == 0 ? &tmA0 : &tmA1;
        const CUtensorMap* mb = pair == 0 ? &tmB0 : &tmB1;
        uint8_t* sa = smem + s * STAGE_BYTES;
        uint8_t* sb = sa + A_STAGE_BYTES;
        if (!p.a_mn) {
          if (lane == 0) tma_load_2d(sa, ma, k0, m0, &full[s]);
        } else if (p.a_3d) {
          if (lane == 0) tma_load_3d(sa, ma, 0, k0, m0 / 32, &full[s]);
        } else if (lane < BM / 32) {
          tma_load_2d(sa + lane * (BK * 128), ma, m0 + 32 * lane, k0, &full[s]);
        }
        if (!p.b_mn) {
          if (lane == 8) tma_load_2d(sb, mb, k0, n0, &full[s]);
        } else if (p.b_3d) {
          if (lane == 8) tma_load_3d(sb, mb, 0, k0, n0 / 32, &full[s]);
        } else if (lane >= 8 && lane < 8 + bn / 32) {
          const int c = lane - 8;
          tma_load_2d(sb + c * (BK * 128), mb, n0 + 32 * c, k0, &full[s]);
        }
      }
    }
  } else if (warp == 1) {
    if (lane == 0) {
      // ---------------------------------------------------------------- MMA issuer
      // instruction descriptor: D = F32, A = B = TF32, majors, N >> 3, M >> 4
      const uint32_t idesc = (1u << 4) | (2u << 7) | (2u << 10) | ((uint32_t)(p.a_mn ? 1 : 0) << 15) |
                             ((uint32_t)(p.b_mn ? 1 : 0) << 16) | ((uint32_t)(bn >> 3) << 17) | ((uint32_t)(BM >> 4) << 24);
      const uint32_t a_lbo = p.a_mn ? BK * 128 : 16, b_lbo = p.b_mn ? BK * 128 : 16;
      const uint32_t a_step = p.a_mn ? 1024 : 32, b_step = p.b_mn ? 1024 : 32;
      const uint32_t a_sbo = p.a_mn ? 512 : 1024, b_sbo = p.b_mn ? 512 : 1024;
      const uint32_t a_lay = p.a_mn ? 1 : 2, b_lay = p.b_mn ? 1 : 2;
      int it = 0, ti = 0;
      bool ok = true;
      for (int t = blockIdx.x; t < p.tiles && ok; t += gridDim.x, ++ti) {
        const int buf = ti & 1;
        const uint32_t aph = (ti >> 1) & 1;
        ok = wait_or_abort(&acc_empty[buf], aph ^ 1, abort_flag, p.err, 4);   // epilogue has drained this accumulator
        if (!ok) break;
        tc_fence_after();
        const uint32_t tmem_d = tmem_base + (uint32_t)(buf * BN_MAX);
        for (int kb = 0; kb < total_kb; ++kb, ++it) {
          const int s = it % STAGES;
          const uint32_t ph = (it / STAGES) & 1;
          ok = wait_or_abort(&full[s], ph, abort_flag, p.err, 2);
          if (!ok) break;
          tc_fence_after();
          const uint32_t sa = smem_u32(smem + s * STAGE_BYTES);
          const uint32_t sb = sa + A_STAGE_BYTES;
#pragma unroll
          for (int k = 0; k < BK / 8; ++k) {
            const uint64_t ad = make_desc(sa + k * a_step, a_lbo, a_sbo, a_lay);
            const uint64_t bd = make_desc(sb + k * b_step, b_lbo, b_sbo, b_lay);
            mma_tf32(tmem_d, ad, bd, idesc, (kb | k) != 0 ? 1u : 0u);
          }
          mma_commit(&empty[s]);  // frees the slot once these MMAs have read it
        }
        if (ok) mma_commit(&acc_full[buf]);
      }
    }
  } else {
    // ------------------------------------------------------------------ epilogue (warps 2..9)
    // Two warps per tensor-memory quadrant; the pair alternates over the tile's 32-column chunks.
    const int quad = warp & 3;            // tensor-memory lanes 32*quad .. 32*quad+31 are this warp's
    const int half = (warp - 2) >> 2;     // 0 or 1: which chunks of the tile this warp takes
    int ti = 0;
    for (int t = blockIdx.x; t < p.tiles; t += gridDim.x, ++ti) {
      const int m0 = (t / p.tiles_n) * BM, n0 = (t % p.tiles_n) * bn;
      const int buf = ti & 1;
      const uint32_t aph = (ti >> 1) & 1;
      int good = 1;
      if (lane == 0) good = wait_or_abort(&acc_full[buf], aph, abort_flag, p.err, 3) ? 1 : 0;
      good = __shfl_sync(0xffffffffu, good, 0);
      if (!good) break;
      tc_fence_after();
      // Registers only: the MMA's operand reads and the TMA writes already use all of the shared-memory
      // bandwidth, so staging the tile through shared memory would starve.  Lane = row; every lane
      // moves 16 bytes per access and a row's 128 bytes are completed by consecutive accesses.
      const int m = m0 + quad * 32 + lane;
      const bool m_ok = m < p.M;
      const float* zrow = p.dsig ? p.dsig + (long long)((m / p.dsig_div) % p.dsig_rows) * p.ld_dsig : nullptr;
      const float* crow = p.cin ? p.cin + (long long)m * p.ld_cin : nullptr;
      float* drow = p.D + (long long)m * p.ldd;
      for (int c = half; c < bn / 32; c += 2) {
        const int nb = n0 + c * 32;
        if (nb >= p.N) break;               // warp-uniform
        const bool full = p.vec_epi && nb + 32 <= p.N;   // warp-uniform: whole chunk in range and 16-byte aligned
        float4 zc[8], ci[8];
        if (full && m_ok) {                 // all global reads of the chunk in flight before anything waits
#pragma unroll
          for (int q = 0; q < 8; ++q) {
            zc[q] = zrow ? __ldg(reinterpret_cast<const float4*>(zrow + nb) + q) : make_float4(0.f, 0.f, 0.f, 0.f);
            ci[q] = crow ? __ldg(reinterpret_cast<const float4*>(crow + nb) + q) : make_float4(0.f, 0.f, 0.f, 0.f);
          }
        }
        float v[32];
        tmem_ld32(tmem_base + ((uint32_t)(quad * 32) << 16) + (uint32_t)(buf * BN_MAX + c * 32), v);
        if (!m_ok) continue;
        if (full) {
#pragma unroll
          for (int q = 0; q < 8; ++q) {
            float4 bz = make_float4(0.f, 0.f, 0.f, 0.f);
            if (p.bias) bz = __ldg(reinterpret_cast<const float4*>(p.bias + nb) + q);
            float x[4] = {v[4 * q] + bz.x, v[4 * q + 1] + bz.y, v[4 * q + 2] + bz.z, v[4 * q + 3] + bz.w};
            const float z[4] = {zc[q].x, zc[q].y, zc[q].z, zc[q].w};
            const float cc[4] = {ci[q].x, ci[q].y, ci[q].z, ci[q].w};
#pragma unroll
            for (int j = 0; j < 4; ++j) {
              if (p.sigmoid) x[j] = 1.f / (1.f + __expf(-x[j]));
              if (zrow) x[j] *= z[j] * (1.f - z[j]);
              x[j] *= p.alpha;
              if (crow) x[j] = fmaf(p.beta, cc[j], x[j]);
            }
            reinterpret_cast<float4*>(drow + nb)[q] = make_float4(x[0], x[1], x[2], x[3]);
          }
        } else {                             // ragged or unaligned chunk: element by element
#pragma unroll
          for (int j = 0; j < 32; ++j) {
            const int n = nb + j;
            if (n < p.N) {
              float x = v[j] + (p.bias ? __ldg(p.bias + n) : 0.f);
              if (p.sigmoid) x = 1.f / (1.f + __expf(-x));
              if (zrow) { const float z = __ldg(zrow + n); x *= z * (1.f - z); }
              x *= p.alpha;
              if (crow) x = fmaf(p.beta, __ldg(crow + n), x);
              drow[n] = x;
            }
          }
        }
      }
      // this warp has read its quadrant of the accumulator: let the MMA issuer reuse it
      tc_fence_before();
      __syncwarp();
      if (lane == 0) mbar_arrive(&acc_empty[buf]);
    }
  }
  tc_fence_before();
  __syncthreads();
  if (warp == 2) {
    tc_fence_after();
    asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem_base), "r"(512) : "memory");
  }
}

// ------------------------------------------------------------------------------------------------
// Two-CTA variant: a cluster of two CTAs (two SMs) computes one 256 x bn tile with
// tcgen05.mma.cta_group::2.  CTA r of the pair owns rows [128 r, 128 r + 128) of the tile (its A block
// and its accumulator) and stages half of the B tile (bn/2 rows); the tensor cores of both SMs read
// both halves.  Per k-block each SM therefore moves 16 KB + 16 KB instead of 16 KB + 32 KB through
// shared memory, which is what limits the one-CTA kernel.
// Protocol: both producers wait on their own empty[s] (released in both CTAs by a multicast commit),
// only the leader (rank 0) arms full[s] with the bytes of both CTAs, and both CTAs' TMA loads complete
// on the leader's full[s].  MMAs are issued by the leader only.  acc_full[b] is multicast to both
// CTAs; all 16 epilogue warps of the pair arrive on the leader's acc_empty[b].
//
// Work list: with T tiles on P pairs, pair q runs tiles q, q + P, ... for the floor(T / P) full waves, so
// that all pairs move through neighbouring tiles together (tiles of one A panel are read at the same
// time and hit in L2).  The T mod P tiles left over are each cut along K into up to 16 slices, one per
// pair, and a pair does its slice before its whole tiles.  The pairs of a sliced tile store their raw
// accumulators in a workspace, count themselves in on the tile's flag, wait (bounded) until all slices
// have arrived, and then each sums one share of the tile's column chunks over all slices, in slice
// order, and runs the epilogue on it - all of this on the epilogue warps while the MMA issuer is already
// working on the pair's first whole tile in the other accumulator.  The order of every sum is fixed, so
// results are deterministic.
__device__ __forceinline__ uint32_t cluster_ctarank() {
  uint32_t r;
  asm volatile("mov.u32 %0, %%cluster_ctarank;" : "=r"(r));
  return r;
}
__device__ __forceinline__ uint32_t map_to_cta(uint32_t local_smem_addr, uint32_t rank) {
  uint32_t r;
  asm volatile("mapa.shared::cluster.u32 %0, %1, %2;" : "=r"(r) : "r"(local_smem_addr), "r"(rank));
  return r;
}
// Cluster-wide barrier.  Warps may arrive here after divergent role code, so they reconverge first
// and the non-aligned forms are used.
__device__ __forceinline__ void cluster_sync_all() {
  __syncwarp();
  asm volatile("barrier.cluster.arrive.release;" ::: "memory");
  asm volatile("barrier.cluster.wait.acquire;" ::: "memory");
}
__device__ __forceinline__ void mbar_arrive_cluster(uint32_t cluster_addr) {
  asm volatile("mbarrier.arrive.release.cluster.shared::cluster.b64 _, [%0];" ::"r"(cluster_addr) : "memory");
}
__device__ __forceinline__ void tma2_load_2d(void* dst, const CUtensorMap* map, int x, int y, uint32_t bar_cluster_addr) {
  asm volatile(
      "cp.async.bulk.tensor.2d.cta_group::2.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%2, %3}], [%4];"
      ::"r"(smem_u32(dst)), "l"(reinterpret_cast<uint64_t>(map)), "r"(x), "r"(y), "r"(bar_cluster_addr)
      : "memory");
}
__device__ __forceinline__ void tma2_load_3d(void* dst, const CUtensorMap* map, int x, int y, int z, uint32_t bar_cluster_addr) {
  asm volatile(
      "cp.async.bulk.tensor.3d.cta_group::2.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%2, %3, %4}], [%5];"
      ::"r"(smem_u32(dst)), "l"(reinterpret_cast<uint64_t>(map)), "r"(x), "r"(y), "r"(z), "r"(bar_cluster_addr)
      : "memory");
}
__device__ __forceinline__ void mma2_tf32(uint32_t tmem_d, uint64_t adesc, uint64_t bdesc, uint32_t idesc, uint32_t accum) {
  asm volatile(
      "{\n\t.reg .pred p;\n\t"
      "setp.ne.b32 p, %4, 0;\n\t"
      "tcgen05.mma.cta_group::2.kind::tf32 [%0], %1, %2, %3, p;\n\t}"
      ::"r"(tmem_d), "l"(adesc), "l"(bdesc), "r"(idesc), "r"(accum) : "memory");
}
// commit of the pair's MMAs, arriving on the barrier at this offset in both CTAs
__device__ __forceinline__ void mma2_commit_both(uint64_t* bar) {
  const uint16_t mask = 3;
  asm volatile("tcgen05.commit.cta_group::2.mbarrier::arrive::one.shared::cluster.multicast::cluster.b64 [%0], %1;"
               ::"r"(smem_u32(bar)), "h"(mask) : "memory");
}

struct Work { int prob, tile, kb0, kb1, sliced; };

// idx-th piece of work of CTA pair `pair` (see Tf32Params and GroupParams); false when the pair has no more.
// A single problem whose left-over tiles are cut along K: the pair does its slice FIRST; the store of the partial
// accumulator, the wait for the other slices and the fix-up epilogue then run on the epilogue warps underneath the
// MMAs of the pair's first whole tile instead of being exposed at the end of the kernel.
__device__ __forceinline__ bool next_work(const GroupParams& gp, int pair, int idx, Work& w) {
  if (gp.pr[0].slices >= 2) {                  // (only ever set for a launch with one problem)
    const Tf32Params& p = gp.pr[0];
    const int total_kb = p.kblocks[0] + p.kblocks[1];
    w.prob = 0;
    if (pair < p.rem * p.slices) {
      if (idx == 0) {
        const int j = pair / p.slices, sl = pair - j * p.slices;
        w.tile = p.waves * p.P + j;
        w.kb0 = (int)((long long)total_kb * sl / p.slices);
        w.kb1 = (int)((long long)total_kb * (sl + 1) / p.slices);
        w.sliced = 1;
        return true;
      }
      --idx;
    }
    if (idx >= p.waves) return false;
    w.tile = idx * p.P + pair; w.kb0 = 0; w.kb1 = total_kb; w.sliced = 0;
    return true;
  }
  for (int g = 0; g < gp.n_prob; ++g) {
    const Tf32Params& p = gp.pr[g];
    const int r0 = gp.rstart[g][pair], n_rem = gp.rstart[g][pair + 1] - r0;
    if (idx < p.waves + n_rem) {
      w.prob = g; w.kb0 = 0; w.kb1 = p.kblocks[0] + p.kblocks[1]; w.sliced = 0;
      w.tile = idx < p.waves ? idx * p.P + pair : p.waves * p.P + r0 + (idx - p.waves);
      return true;
    }
    idx -= p.waves + n_rem;
  }
  return false;
}

// Epilogue of one whole, 16-byte-aligned 32 x 32 chunk of a warp's quadrant in the fragment layout of
// tmem_ld_16x256b_x4: value v[4j + 2e + i] of half h is element (row 16h + 8e + lane / 4, column 8j + 2 (lane % 4) + i).
// The epilogue warps are few (two per scheduler) and run beside the main loop, so what bounds them is their own
// instruction stream, not the memory system: the same chunk took 10.7 us with every option tested per element
// and 3.6 us as a plain store.  MODE fixes the options at compile time: 0 = alpha * acc (+ bias), 1 = sigmoid,
// 2 = times the sigmoid derivative of `dsig`, 3 = plus beta * cin; 4 = any combination, tested at run time (its operands
// are read where they are used, so that it needs no more registers than the others: the kernel is at its limit
// of 168 and a spill here would be paid by every mode).
struct EpiArgs {
  const float* dsig; const float* cin; const float* bias; float* D;
  long long ldd, ld_dsig, ld_cin;
  int dsig_rows, dsig_div;   // row m of the tile reads row (m / dsig_div) % dsig_rows of dsig ...
  int dsig_direct;           // ... which is m itself when dsig_div == 1 and dsig_rows >= M (no division per row)
  float alpha, beta;
  int M, sigm;
};

__device__ __forceinline__ long long dsig_row(const EpiArgs& a, int m) {
  return a.dsig_direct ? m : (m / a.dsig_div) % a.dsig_rows;
}

template <int MODE>
__device__ __forceinline__ void epilogue_full_chunk(const EpiArgs& a, uint32_t taddr, int mq, int nb, int lane,
                                                    const float* ws, int slices) {
  const bool use_sigm = MODE == 4 ? a.sigm != 0 : MODE == 1;
  const bool use_dsig = MODE == 4 ? a.dsig != nullptr : MODE == 2;
  const bool use_cin = MODE == 4 ? a.cin != nullptr : MODE == 3;
  float2 op[2][8];                             // [h][4e + j]: the chunk of dsig (mode 2) or of cin (mode 3)
  if (MODE == 2 || MODE == 3) {                // all global reads of the chunk in flight before anything waits
#pragma unroll
    for (int h = 0; h < 2; ++h)
#pragma unroll
      for (int e = 0; e < 2; ++e) {
        const int m = mq + 16 * h + 8 * e;
        const float* row = nullptr;
        if (m < a.M) row = MODE == 3 ? a.cin + (long long)m * a.ld_cin + nb
                                     : a.dsig + dsig_row(a, m) * a.ld_dsig + nb;
#pragma unroll
        for (int j = 0; j < 4; ++j) {
          float2 x = make_float2(0.f, 0.f);
          // (cin: L2-coherent read, in a chained launch it may have been written by another pair of this very launch)
          if (row) x = MODE == 3 ? __ldcg(reinterpret_cast<const float2*>(row + 8 * j)) : __ldg(reinterpret_cast<const float2*>(row + 8 * j));
          op[h][4 * e + j] = x;
        }
      }
  }
  float2 bz[4];
#pragma unroll
  for (int j = 0; j < 4; ++j) bz[j] = a.bias ? __ldg(reinterpret_cast<const float2*>(a.bias + nb + 8 * j)) : make_float2(0.f, 0.f);
#pragma unroll
  for (int h = 0; h < 2; ++h) {                // one 16-row half of the chunk at a time (16 accumulator registers live)
    float v[16];
    if (slices == 0) {
      tmem_ld_16x256b_x4(taddr + ((uint32_t)(16 * h) << 16), v);
      tmem_ld_wait();
    } else {                                   // a tile cut along K: sum of the slices' partials, slice 0 first
#pragma unroll
      for (int i = 0; i < 16; ++i) v[i] = 0.f;
      for (int s2 = 0; s2 < slices; ++s2) {
        const float* wsr = ws + (long long)s2 * (2 * BM * BN_MAX) + (16 * h) * BN_MAX;
#pragma unroll
        for (int e = 0; e < 2; ++e)
#pragma unroll
          for (int j = 0; j < 4; ++j) {
            const float2 x = __ldcg(reinterpret_cast<const float2*>(wsr + (8 * e) * BN_MAX + 8 * j));
            v[4 * j + 2 * e] += x.x; v[4 * j + 2 * e + 1] += x.y;
          }
      }
    }
#pragma unroll
    for (int e = 0; e < 2; ++e) {
      const int m = mq + 16 * h + 8 * e;
      if (m >= a.M) continue;
      float* drow = a.D + (long long)m * a.ldd + nb;
      const float* crow = (MODE == 4 && use_cin) ? a.cin + (long long)m * a.ld_cin + nb : nullptr;
      const float* zrow = (MODE == 4 && use_dsig) ? a.dsig + dsig_row(a, m) * a.ld_dsig + nb : nullptr;
#pragma unroll
      for (int j = 0; j < 4; ++j) {
        float x0 = v[4 * j + 2 * e] + bz[j].x, x1 = v[4 * j + 2 * e + 1] + bz[j].y;
        if (use_sigm) { x0 = 1.f / (1.f + __expf(-x0)); x1 = 1.f / (1.f + __expf(-x1)); }
        if (use_dsig) {
          const float2 z = MODE == 4 ? __ldg(reinterpret_cast<const float2*>(zrow + 8 * j)) : op[h][4 * e + j];
          x0 *= z.x * (1.f - z.x); x1 *= z.y * (1.f - z.y);
        }
        x0 *= a.alpha; x1 *= a.alpha;
        if (MODE == 3) {
          const float2 cc = op[h][4 * e + j];
          x0 = fmaf(a.beta, cc.x, x0); x1 = fmaf(a.beta, cc.y, x1);
        } else if (MODE == 4 && use_cin) {
          const float2 cc = __ldcg(reinterpret_cast<const float2*>(crow + 8 * j));
          x0 = fmaf(a.beta, cc.x, x0); x1 = fmaf(a.beta, cc.y, x1);
        }
        *reinterpret_cast<float2*>(drow + 8 * j) = make_float2(x0, x1);
      }
    }
  }
}

constexpr int B2_STAGE_MAX = (BN_MAX / 2) * BK * 4;          // 16 KB: this CTA's half of the B tile
constexpr int STAGE2_BYTES = A_STAGE_BYTES + B2_STAGE_MAX;   // 32 KB

template <int STAGES>
__global__ void __cluster_dims__(2, 1, 1) __launch_bounds__(320, 1)
gemm_tf32_2cta_kernel(const __grid_constant__ GroupMaps gm, const __grid_constant__ GroupParams gp) {
  extern __shared__ uint8_t smem_raw[];
  uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~(uintptr_t)1023);
  uint64_t* full = reinterpret_cast<uint64_t*>(smem + STAGES * STAGE2_BYTES);
  uint64_t* empty = full + STAGES;
  uint64_t* acc_full = empty + STAGES;   // [2]
  uint64_t* acc_empty = acc_full + 2;    // [2]
  uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(acc_empty + 2);
  volatile int* abort_flag = reinterpret_cast<volatile int*>(tmem_slot + 1);

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const uint32_t rank = cluster_ctarank();
  const int pair = blockIdx.x >> 1;
  int* const err = gp.pr[0].err;

  if (threadIdx.x == 0) {
    for (int s = 0; s < STAGES; ++s) { mbar_init(&full[s], 1); mbar_init(&empty[s], 1); }
    for (int b = 0; b < 2; ++b) { mbar_init(&acc_full[b], 1); mbar_init(&acc_empty[b], 16); }
    *abort_flag = 0;
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  if (warp == 2) {  // both CTAs of the pair allocate all 512 columns, same warp, same destination offset
    asm volatile("tcgen05.alloc.cta_group::2.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(tmem_slot)), "r"(512) : "memory");
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::2.sync.aligned;" ::: "memory");
  }
  tc_fence_before();
  cluster_sync_all();      // barriers of both CTAs are initialised before anyone signals across the pair
  tc_fence_after();
  const uint32_t tmem_base = *tmem_slot;
  grid_dep_wait();
  grid_dep_launch();

  if (warp == 0) {
    // ------------------------------------------------------------------ producer (both CTAs)
    int it = 0;
    bool ok = true;
    Work w;
    for (int wi = 0; ok && next_work(gp, pair, wi, w); ++wi) {
      const Tf32Params& p = gp.pr[w.prob];
      const int bn = p.bn, hb = p.bn >> 1;                     // hb: B rows staged by each CTA
      const uint32_t pair_tx = 2u * (A_STAGE_BYTES + (uint32_t)hb * BK * 4);
      const int t = w.tile, kb0 = w.kb0, kb1 = w.kb1;
      const int m0 = (t / p.tiles_n) * (2 * BM) + (int)rank * BM;
      const int n0 = (t % p.tiles_n) * bn + (int)rank * hb;
      if (gp.dep_prob[w.prob] >= 0) {
        // an operand of this tile is written by an earlier problem of this launch: wait until its tiles are stored
        const int d = gp.dep_prob[w.prob];
        const int* ctr = gp.done + (long long)d * gp.done_stride + (gp.dep_all[w.prob] ? gp.done_stride - 1 : t / p.tiles_n);
        const int want = 16 * (gp.dep_all[w.prob] ? gp.pr[d].tiles : gp.pr[d].tiles_n);
        int good = 1;
        if (lane == 0) {
          const unsigned long long t0 = globaltimer();
          while (ld_acquire_gpu(ctr) < want) {
            if (*abort_flag || globaltimer() - t0 > WAIT_LIMIT_NS) { atomicCAS(err, 0, 6); *abort_flag = 1; good = 0; break; }
            __nanosleep(100);
          }
        }
        good = __shfl_sync(0xffffffffu, good, 0);
        if (!good) { ok = false; break; }
        asm volatile("fence.proxy.async.global;" ::: "memory");   // the stores were generic, the loads below are TMA's
        __syncwarp();
      }
      for (int kb = kb0; kb < kb1; ++kb, ++it) {
        const int s = it % STAGES;
        const uint32_t ph = (it / STAGES) & 1;
        int good = 1;
        if (lane == 0) good = wait_or_abort(&empty[s], ph ^ 1, abort_flag, err, 1) ? 1 : 0;
        good = __shfl_sync(0xffffffffu, good, 0);
        if (!good) { ok = false; break; }
        if (rank == 0 && lane == 0) mbar_expect_tx(&full[s], pair_tx);
        __syncwarp();
        const uint32_t full_leader = map_to_cta(smem_u32(&full[s]), 0);
        const int pr = kb < p.kblocks[0] ? 0 : 1;
        const int k0 = (pr == 0 ? kb : kb - p.kblocks[0]) * BK;
        const CUtensorMap* ma = &gm.m[w.prob][2 * pr];
        const CUtensorMap* mb = &gm.m[w.prob][2 * pr + 1];
        uint8_t* sa = smem + s * STAGE2_BYTES;
        uint8_t* sb = sa + A_STAGE_BYTES;
        if (!p.a_mn) {
          if (lane == 0) tma2_load_2d(sa, ma, k0, m0, full_leader);
        } else if (p.a_3d) {
          if (lane == 0) tma2_load_3d(sa, ma, 0, k0, m0 / 32, full_leader);
        } else if (lane < BM / 32) {
          tma2_load_2d(sa + lane * (BK * 128), ma, m0 + 32 * lane, k0, full_leader);
        }
        if (!p.b_mn) {
          if (lane == 8) tma2_load_2d(sb, mb, k0, n0, full_leader);
        } else if (p.b_3d) {
          if (lane == 8) tma2_load_3d(sb, mb, 0, k0, n0 / 32, full_leader);
        } else if (lane >= 8 && lane < 8 + hb / 32) {
          const int c = lane - 8;
          tma2_load_2d(sb + c * (BK * 128), mb, n0 + 32 * c, k0, full_leader);
        }
      }
    }
  } else if (warp == 1) {
    if (rank == 0 && lane == 0) {
      // ---------------------------------------------------------------- MMA issuer (leader CTA only)
      int it = 0, ti = 0;
      bool ok = true;
      Work w;
      for (int wi = 0; ok && next_work(gp, pair, wi, w); ++wi, ++ti) {
        const Tf32Params& p = gp.pr[w.prob];
        const uint32_t idesc = (1u << 4) | (2u << 7) | (2u << 10) | ((uint32_t)(p.a_mn ? 1 : 0) << 15) |
                               ((uint32_t)(p.b_mn ? 1 : 0) << 16) | ((uint32_t)(p.bn >> 3) << 17) | ((uint32_t)((2 * BM) >> 4) << 24);
        const uint32_t a_lbo = p.a_mn ? BK * 128 : 16, b_lbo = p.b_mn ? BK * 128 : 16;
        const uint32_t a_step = p.a_mn ? 1024 : 32, b_step = p.b_mn ? 1024 : 32;
        const uint32_t a_sbo = p.a_mn ? 512 : 1024, b_sbo = p.b_mn ? 512 : 1024;
        const uint32_t a_lay = p.a_mn ? 1 : 2, b_lay = p.b_mn ? 1 : 2;
        const int kb0 = w.kb0, kb1 = w.kb1;
        const int buf = ti & 1;
        const uint32_t aph = (ti >> 1) & 1;
        ok = wait_or_abort(&acc_empty[buf], aph ^ 1, abort_flag, err, 4);
        if (!ok) break;
        tc_fence_after();
        const uint32_t tmem_d = tmem_base + (uint32_t)(buf * BN_MAX);
        for (int kb = kb0; kb < kb1; ++kb, ++it) {
          const int s = it % STAGES;
          const uint32_t ph = (it / STAGES) & 1;
          ok = wait_or_abort(&full[s], ph, abort_flag, err, 2);
          if (!ok) break;
          tc_fence_after();
          const uint32_t sa = smem_u32(smem + s * STAGE2_BYTES);
          const uint32_t sb = sa + A_STAGE_BYTES;
#pragma unroll
          for (int k = 0; k < BK / 8; ++k) {
            const uint64_t ad = make_desc(sa + k * a_step, a_lbo, a_sbo, a_lay);
            const uint64_t bd = make_desc(sb + k * b_step, b_lbo, b_sbo, b_lay);
            mma2_tf32(tmem_d, ad, bd, idesc, (kb > kb0 || k != 0) ? 1u : 0u);
          }
          mma2_commit_both(&empty[s]);
        }
        if (ok) mma2_commit_both(&acc_full[buf]);
      }
    }
  } else {
    // ------------------------------------------------------------------ epilogue (warps 2..9, both CTAs)
    // Fragment layout of tmem_ld_16x256b_x4: this thread's 32 values of a 32 x 32 chunk are v[h][4j + 2e + i] =
    // element (row 16h + 8e + lane/4, column 8j + 2 (lane%4) + i) of the warp's quadrant.
    const int quad = warp & 3;
    const int half = (warp - 2) >> 2;
    const int rsub = lane >> 2, csub = (lane & 3) * 2;
    int ti = 0;
    Work w;
    for (int wi = 0; next_work(gp, pair, wi, w); ++wi, ++ti) {
      const Tf32Params& p = gp.pr[w.prob];
      const int bn = p.bn;
      const int t = w.tile;
      const int m0 = (t / p.tiles_n) * (2 * BM) + (int)rank * BM, n0 = (t % p.tiles_n) * bn;
      const int buf = ti & 1;
      const uint32_t aph = (ti >> 1) & 1;
      int good = 1;
      if (lane == 0) good = wait_or_abort(&acc_full[buf], aph, abort_flag, err, 3) ? 1 : 0;
      good = __shfl_sync(0xffffffffu, good, 0);
      if (!good) break;
      tc_fence_after();
      const int n_chunks = min(bn / 32, (p.N - n0 + 31) / 32);   // column chunks of this tile that exist
      const uint32_t tq = tmem_base + ((uint32_t)(quad * 32) << 16) + (uint32_t)(buf * BN_MAX);
      int sl = 0, grp = 0;                                       // slice index and first pair of the tile's group
      if (w.sliced) {
        grp = (pair / p.slices) * p.slices;
        sl = pair - grp;
        // 1. raw accumulator of this slice to the workspace slot of this pair
        float* wsw = p.sk_ws + (((long long)pair * 2 + rank) * BM + quad * 32 + rsub) * BN_MAX + csub;
        for (int c = half; c < n_chunks; c += 2) {
          float v[2][16];
          tmem_ld_16x256b_x4(tq + (uint32_t)(c * 32), v[0]);
          tmem_ld_16x256b_x4(tq + (16u << 16) + (uint32_t)(c * 32), v[1]);
          tmem_ld_wait();
#pragma unroll
          for (int h = 0; h < 2; ++h)
#pragma unroll
            for (int e = 0; e < 2; ++e)
#pragma unroll
              for (int j = 0; j < 4; ++j)
                __stcg(reinterpret_cast<float2*>(wsw + (long long)(16 * h + 8 * e) * BN_MAX + c * 32 + 8 * j),
                       make_float2(v[h][4 * j + 2 * e], v[h][4 * j + 2 * e + 1]));
        }
        // the accumulator is free again; the tensor pipe has no further use for it in this pair
        tc_fence_before();
        __threadfence();
        __syncwarp();
        if (lane == 0) {
          mbar_arrive_cluster(map_to_cta(smem_u32(&acc_empty[buf]), 0));
          int* flag_w = p.sk_flags + pair / p.slices;
          atomicAdd(flag_w, 1);
          // 2. wait until the 16 warps of every slice of this tile have stored theirs
          const volatile int* flag = flag_w;
          const int want = 16 * p.slices;
          const unsigned long long t0 = globaltimer();
          while (*flag < want) {
            if (*abort_flag || globaltimer() - t0 > WAIT_LIMIT_NS) { atomicCAS(err, 0, 5); *abort_flag = 1; good = 0; break; }
            __nanosleep(200);   // sixteen warps per pair poll the same word: keep them off the L2 while the pair's MMAs run
          }
          __threadfence();
          // 3. count out again: the last of the tile's warps to have seen the full count puts the flag back to
          // zero for the next launch (no memset between launches; the count only grows until then, so nobody
          // still waiting can miss it)
          if (good && atomicAdd(flag_w, 1) == 2 * want - 1) *reinterpret_cast<volatile int*>(flag_w) = 0;
        }
        good = __shfl_sync(0xffffffffu, good, 0);
        if (!good) break;
      }
      {
        const int mq = m0 + quad * 32 + rsub;                    // this thread's rows are mq + 16h + 8e
        EpiArgs ea;
        ea.dsig = p.dsig; ea.cin = p.cin; ea.bias = p.bias; ea.D = p.D;
        ea.ldd = p.ldd; ea.ld_dsig = p.ld_dsig; ea.ld_cin = p.ld_cin;
        ea.dsig_rows = p.dsig_rows; ea.dsig_div = p.dsig_div;
        ea.dsig_direct = p.dsig_div == 1 && p.dsig_rows >= p.M;
        ea.alpha = p.alpha; ea.beta = p.beta; ea.M = p.M; ea.sigm = p.sigmoid;
        const int N = p.N, vec_epi = p.vec_epi;
        const int n_opt = (p.sigmoid ? 1 : 0) + (p.dsig ? 1 : 0) + (p.cin ? 1 : 0);
        const int mode = n_opt == 0 ? 0 : n_opt > 1 ? 4 : p.sigmoid ? 1 : p.dsig ? 2 : 3;
        // whole tile: this warp's chunks are half, half + 2, ...; sliced tile: the pair's share of the
        // chunks is sl, sl + slices, ..., dealt alternately to the two warps of a quadrant
        const int c_first = w.sliced ? sl + half * p.slices : half;
        const int c_step = w.sliced ? 2 * p.slices : 2;
        const int n_slices = w.sliced ? p.slices : 0;
        const float* const ws0 = w.sliced ? p.sk_ws + (((long long)grp * 2 + rank) * BM + quad * 32 + rsub) * BN_MAX + csub : nullptr;
        for (int c = c_first; c < n_chunks; c += c_step) {
          const int nb = n0 + c * 32 + csub;                     // this thread's columns are nb + 8j, nb + 8j + 1
          const uint32_t taddr = tq + (uint32_t)(c * 32);
          if (vec_epi && n0 + c * 32 + 32 <= N) {                // warp-uniform: whole chunk in range, 16-byte aligned rows
            const float* ws = ws0 + c * 32;
            switch (mode) {
              case 0: epilogue_full_chunk<0>(ea, taddr, mq, nb, lane, ws, n_slices); break;
              case 1: epilogue_full_chunk<1>(ea, taddr, mq, nb, lane, ws, n_slices); break;
              case 2: epilogue_full_chunk<2>(ea, taddr, mq, nb, lane, ws, n_slices); break;
              case 3: epilogue_full_chunk<3>(ea, taddr, mq, nb, lane, ws, n_slices); break;
              default: epilogue_full_chunk<4>(ea, taddr, mq, nb, lane, ws, n_slices); break;
            }
            continue;
          }
          // ragged or unaligned chunk: element by element
#pragma unroll 1
          for (int h = 0; h < 2; ++h) {
            float v[16];
            if (!w.sliced) {
              tmem_ld_16x256b_x4(taddr + ((uint32_t)(16 * h) << 16), v);
              tmem_ld_wait();
            } else {
#pragma unroll
              for (int i = 0; i < 16; ++i) v[i] = 0.f;
              for (int s2 = 0; s2 < n_slices; ++s2) {
                const float* wsr = ws0 + c * 32 + (long long)s2 * (2 * BM * BN_MAX) + (16 * h) * BN_MAX;
#pragma unroll
                for (int e = 0; e < 2; ++e)
#pragma unroll
                  for (int j = 0; j < 4; ++j) {
                    const float2 x = __ldcg(reinterpret_cast<const float2*>(wsr + (8 * e) * BN_MAX + 8 * j));
                    v[4 * j + 2 * e] += x.x; v[4 * j + 2 * e + 1] += x.y;
                  }
              }
            }
#pragma unroll
            for (int e = 0; e < 2; ++e) {
              const int m = mq + 16 * h + 8 * e;
              if (m >= ea.M) continue;
              const float* zrow = ea.dsig ? ea.dsig + dsig_row(ea, m) * ea.ld_dsig : nullptr;
              const float* crow = ea.cin ? ea.cin + (long long)m * ea.ld_cin : nullptr;
              float* drow = ea.D + (long long)m * ea.ldd;
#pragma unroll
              for (int j = 0; j < 4; ++j)
#pragma unroll
                for (int i = 0; i < 2; ++i) {
                  const int n = nb + 8 * j + i;
                  if (n < N) {
                    float x = v[4 * j + 2 * e + i] + (ea.bias ? __ldg(ea.bias + n) : 0.f);
                    if (ea.sigm) x = 1.f / (1.f + __expf(-x));
                    if (zrow) { const float z = __ldg(zrow + n); x *= z * (1.f - z); }
                    x *= ea.alpha;
                    if (crow) x = fmaf(ea.beta, __ldcg(crow + n), x);
                    drow[n] = x;
                  }
                }
            }
          }
        }
      }
      if (!w.sliced) {       // (a sliced tile released its accumulator right after storing it)
        tc_fence_before();
        __syncwarp();
        if (lane == 0) mbar_arrive_cluster(map_to_cta(smem_u32(&acc_empty[buf]), 0));
      }
      if (gp.signal[w.prob]) {
        // a later problem of this launch reads this tile: publish this warp's stores, then count the warp in
        __threadfence();
        asm volatile("fence.proxy.async.global;" ::: "memory");
        __syncwarp();
        if (lane == 0) {
          int* base = gp.done + (long long)w.prob * gp.done_stride;
          if (gp.signal[w.prob] & 1) atomicAdd(base + t / p.tiles_n, 1);
          if (gp.signal[w.prob] & 2) atomicAdd(base + gp.done_stride - 1, 1);
        }
      }
    }
  }
  tc_fence_before();
  cluster_sync_all();      // neither CTA leaves (or frees tensor memory) while the other may still use it
  if (warp == 2) {
    tc_fence_after();
    asm volatile("tcgen05.dealloc.cta_group::2.sync.aligned.b32 %0, %1;" ::"r"(tmem_base), "r"(512) : "memory");
  }
}

// ------------------------------------------------------------------------------------------------
// Error-compensated variant (FP32-accurate results from the TF32 tensor cores).
// Every operand X arrives as two matrices X = Xhi + Xlo, both exactly representable in TF32.  A logical
// product A B is computed as Alo Bhi + Ahi Blo + Ahi Bhi: a ring slot holds the hi and lo tiles of both
// operands for one k-block (64 KB per CTA) and every K = 8 step issues the three products, small terms
// first, so each operand byte is fetched once for three MMAs.  The tensor core adds into its FP32
// accumulator with truncation (measured: a relative bias of about 1e-9 per unit of K in a plain TF32
// accumulation), so the K range is cut into chunks of xp.chunk_kb k-blocks; each chunk is accumulated in
// tensor memory on its own (the two 256-column accumulators alternate per chunk) and the epilogue warps add
// the chunks into a running sum held in registers, in FP32 with round-to-nearest.  That needs 128 registers per epilogue thread for the sums
// alone, so the block has three warpgroups and moves registers between them:
//   warps 0..3   (56 registers)   0 = TMA producer, 1 = MMA issuer, 2 = tensor-memory allocation, 3 idle
//   warps 4..11  (224 registers)  epilogue, two warps per 32-lane quadrant of tensor memory
// Whole tiles only, in wave order (no K slices).  Same pair protocol as the kernel above.
constexpr int MAX_PAIRS = 2;                          // logical operand pairs accumulated into one tile
constexpr int X3_THREADS = 384;
constexpr int X3_STAGES = 3;
constexpr int X3_STAGE_BYTES = 2 * STAGE2_BYTES;      // 64 KB: A hi, A lo, B-half hi, B-half lo
constexpr int X3_REGS_LOW = 56, X3_REGS_HIGH = 224;   // 128 * 56 + 256 * 224 = 384 * 168

struct MapSet { CUtensorMap a_hi[MAX_PAIRS], a_lo[MAX_PAIRS], b_hi[MAX_PAIRS], b_lo[MAX_PAIRS]; };

struct X3Params {
  int n_pairs;
  int kblocks[MAX_PAIRS];
  int chunk_kb;
};

// One whole, 16-byte-aligned chunk of 32 finished sums of a row (lane = row) through the epilogue options and out,
// with the options fixed at compile time as in epilogue_full_chunk: 0 = alpha * sum (+ bias), 1 = sigmoid,
// 2 = times the sigmoid derivative of zrow, 3 = plus beta * crow, 4 = any combination, tested per element.  In modes
// 2 and 3 the 128 bytes of the operand are requested before the first of them is used (the running sums of the
// other chunks leave room for that one buffer); in mode 4 the loads stay beside their use, two steps at a time.
template <int MODE>
__device__ __forceinline__ void x3_store_chunk(const Tf32Params& p, const float* run, const float* zrow, const float* crow,
                                               float* drow, int nb, float* hrow, float* lrow) {
  const bool use_sigm = MODE == 4 ? p.sigmoid != 0 : MODE == 1;
  const bool use_dsig = MODE == 4 ? zrow != nullptr : MODE == 2;
  const bool use_cin = MODE == 4 ? crow != nullptr : MODE == 3;
  float4 op[8];
  if (MODE == 2 || MODE == 3) {
    const float4* src = reinterpret_cast<const float4*>(MODE == 2 ? zrow : crow);
#pragma unroll
    for (int q = 0; q < 8; ++q) op[q] = __ldg(src + q);
  }
#pragma unroll
  for (int q = 0; q < 8; ++q) {
    float4 bz = make_float4(0.f, 0.f, 0.f, 0.f);
    if (p.bias) bz = __ldg(reinterpret_cast<const float4*>(p.bias + nb) + q);
    float4 o = make_float4(0.f, 0.f, 0.f, 0.f), o2 = o;
    if (MODE == 2 || MODE == 3) o = op[q];
    if (MODE == 4 && use_dsig) o = __ldg(reinterpret_cast<const float4*>(zrow) + q);
    if (MODE == 4 && use_cin) o2 = __ldg(reinterpret_cast<const float4*>(crow) + q);
    float x[4] = {run[4 * q] + bz.x, run[4 * q + 1] + bz.y, run[4 * q + 2] + bz.z, run[4 * q + 3] + bz.w};
    const float z[4] = {o.x, o.y, o.z, o.w};
    const float cv[4] = {MODE == 4 ? o2.x : o.x, MODE == 4 ? o2.y : o.y, MODE == 4 ? o2.z : o.z, MODE == 4 ? o2.w : o.w};
#pragma unroll
    for (int e = 0; e < 4; ++e) {
      if (use_sigm) x[e] = 1.f / (1.f + expf(-x[e]));
      if (use_dsig) x[e] *= z[e] * (1.f - z[e]);
      x[e] *= p.alpha;
      if (use_cin) x[e] = fmaf(p.beta, cv[e], x[e]);
    }
    reinterpret_cast<float4*>(drow)[q] = make_float4(x[0], x[1], x[2], x[3]);
    if (hrow) {
      float h[4];
#pragma unroll
      for (int e = 0; e < 4; ++e) { h[e] = round_tf32(x[e]); x[e] = round_tf32(x[e] - h[e]); }
      reinterpret_cast<float4*>(hrow)[q] = make_float4(h[0], h[1], h[2], h[3]);
      reinterpret_cast<float4*>(lrow)[q] = make_float4(x[0], x[1], x[2], x[3]);
    }
    // the running sums leave few registers: keep the loads of at most two steps in flight
    if (MODE == 4 && (q & 1)) asm volatile("" ::: "memory");
  }
}

template <int STAGES>
__global__ void __cluster_dims__(2, 1, 1) __launch_bounds__(X3_THREADS, 1)
gemm_tf32x3_kernel(const __grid_constant__ MapSet maps, const Tf32Params p, const X3Params xp) {
  extern __shared__ uint8_t smem_raw[];
  uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~(uintptr_t)1023);
  uint64_t* full = reinterpret_cast<uint64_t*>(smem + STAGES * X3_STAGE_BYTES);
  uint64_t* empty = full + STAGES;
  uint64_t* acc_full = empty + STAGES;   // [2]
  uint64_t* acc_empty = acc_full + 2;    // [2]
  uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(acc_empty + 2);
  volatile int* abort_flag = reinterpret_cast<volatile int*>(tmem_slot + 1);

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const uint32_t rank = cluster_ctarank();
  const int pair = blockIdx.x >> 1;
  int total_kb = 0;
  for (int i = 0; i < xp.n_pairs; ++i) total_kb += xp.kblocks[i];
  const int n_chunks_k = (total_kb + xp.chunk_kb - 1) / xp.chunk_kb;
  const int bn = p.bn, hb = p.bn >> 1;
  const uint32_t pair_tx = 4u * (A_STAGE_BYTES + (uint32_t)hb * BK * 4);   // two CTAs x (hi + lo) x (A + B half)
  // tiles of this pair: pair, pair + P, ... (whole waves), then one of the `rem` left over
  const int my_tiles = p.waves + (pair < p.rem ? 1 : 0);

  if (threadIdx.x == 0) {
    for (int s = 0; s < STAGES; ++s) { mbar_init(&full[s], 1); mbar_init(&empty[s], 1); }
    for (int b = 0; b < 2; ++b) { mbar_init(&acc_full[b], 1); mbar_init(&acc_empty[b], 16); }
    *abort_flag = 0;
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  if (warp == 2) {
    asm volatile("tcgen05.alloc.cta_group::2.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(tmem_slot)), "r"(512) : "memory");
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::2.sync.aligned;" ::: "memory");
  }
  tc_fence_before();
  cluster_sync_all();
  tc_fence_after();
  const uint32_t tmem_base = *tmem_slot;
  grid_dep_wait();
  grid_dep_launch();

  if (warp < 4) {
    asm volatile("setmaxnreg.dec.sync.aligned.u32 %0;" ::"n"(X3_REGS_LOW));
    if (warp == 0) {
      // ---------------------------------------------------------------- producer (both CTAs)
      int it = 0;
      bool ok = true;
      for (int ti = 0; ti < my_tiles && ok; ++ti) {
        const int t = ti * p.P + pair;
        const int m0 = (t / p.tiles_n) * (2 * BM) + (int)rank * BM;
        const int n0 = (t % p.tiles_n) * bn + (int)rank * hb;
        int pr = 0, kk = 0;                       // operand pair and k-block inside it
        for (int kb = 0; kb < total_kb; ++kb, ++it, ++kk) {
          while (kk >= xp.kblocks[pr]) { kk = 0; ++pr; }
          const int s = it % STAGES;
          const uint32_t ph = (it / STAGES) & 1;
          int good = 1;
          if (lane == 0) good = wait_or_abort(&empty[s], ph ^ 1, abort_flag, p.err, 1) ? 1 : 0;
          good = __shfl_sync(0xffffffffu, good, 0);
          if (!good) { ok = false; break; }
          if (rank == 0 && lane == 0) mbar_expect_tx(&full[s], pair_tx);
          __syncwarp();
          const uint32_t full_leader = map_to_cta(smem_u32(&full[s]), 0);
          const int k0 = kk * BK;
          uint8_t* sa = smem + s * X3_STAGE_BYTES;            // A hi | A lo | B hi | B lo
          uint8_t* sb = sa + 2 * A_STAGE_BYTES;
          if (!p.a_mn) {
            if (lane == 0) tma2_load_2d(sa, &maps.a_hi[pr], k0, m0, full_leader);
            if (lane == 1) tma2_load_2d(sa + A_STAGE_BYTES, &maps.a_lo[pr], k0, m0, full_leader);
          } else {
            if (lane == 0) tma2_load_3d(sa, &maps.a_hi[pr], 0, k0, m0 / 32, full_leader);
            if (lane == 1) tma2_load_3d(sa + A_STAGE_BYTES, &maps.a_lo[pr], 0, k0, m0 / 32, full_leader);
          }
          if (!p.b_mn) {
            if (lane == 8) tma2_load_2d(sb, &maps.b_hi[pr], k0, n0, full_leader);
            if (lane == 9) tma2_load_2d(sb + B2_STAGE_MAX, &maps.b_lo[pr], k0, n0, full_leader);
          } else {
            if (lane == 8) tma2_load_3d(sb, &maps.b_hi[pr], 0, k0, n0 / 32, full_leader);
            if (lane == 9) tma2_load_3d(sb + B2_STAGE_MAX, &maps.b_lo[pr], 0, k0, n0 / 32, full_leader);
          }
        }
      }
    } else if (warp == 1 && rank == 0 && lane == 0) {
      // ---------------------------------------------------------------- MMA issuer (leader CTA only)
      const uint32_t idesc = (1u << 4) | (2u << 7) | (2u << 10) | ((uint32_t)(p.a_mn ? 1 : 0) << 15) |
                             ((uint32_t)(p.b_mn ? 1 : 0) << 16) | ((uint32_t)(bn >> 3) << 17) | ((uint32_t)((2 * BM) >> 4) << 24);
      const uint32_t a_lbo = p.a_mn ? BK * 128 : 16, b_lbo = p.b_mn ? BK * 128 : 16;
      const uint32_t a_step = p.a_mn ? 1024 : 32, b_step = p.b_mn ? 1024 : 32;
      const uint32_t a_sbo = p.a_mn ? 512 : 1024, b_sbo = p.b_mn ? 512 : 1024;
      const uint32_t a_lay = p.a_mn ? 1 : 2, b_lay = p.b_mn ? 1 : 2;
      int it = 0, ci = 0;                          // ring position, running chunk count (accumulator phase)
      bool ok = true;
      for (int ti = 0; ti < my_tiles && ok; ++ti) {
        for (int ch = 0; ch < n_chunks_k && ok; ++ch, ++ci) {
          const int kb0 = ch * xp.chunk_kb, kb1 = min(total_kb, kb0 + xp.chunk_kb);
          const int buf = ci & 1;
          const uint32_t aph = (ci >> 1) & 1;
          ok = wait_or_abort(&acc_empty[buf], aph ^ 1, abort_flag, p.err, 4);
          if (!ok) break;
          tc_fence_after();
          const uint32_t tmem_d = tmem_base + (uint32_t)(buf * BN_MAX);
          for (int kb = kb0; kb < kb1; ++kb, ++it) {
            const int s = it % STAGES;
            const uint32_t ph = (it / STAGES) & 1;
            ok = wait_or_abort(&full[s], ph, abort_flag, p.err, 2);
            if (!ok) break;
            tc_fence_after();
            const uint32_t sa = smem_u32(smem + s * X3_STAGE_BYTES);
            const uint32_t sb = sa + 2 * A_STAGE_BYTES;
#pragma unroll
            for (int k = 0; k < BK / 8; ++k) {
              const uint64_t ah = make_desc(sa + k * a_step, a_lbo, a_sbo, a_lay);
              const uint64_t al = make_desc(sa + A_STAGE_BYTES + k * a_step, a_lbo, a_sbo, a_lay);
              const uint64_t bh = make_desc(sb + k * b_step, b_lbo, b_sbo, b_lay);
              const uint64_t bl = make_desc(sb + B2_STAGE_MAX + k * b_step, b_lbo, b_sbo, b_lay);
              mma2_tf32(tmem_d, al, bh, idesc, (kb > kb0 || k != 0) ? 1u : 0u);   // small terms first
              mma2_tf32(tmem_d, ah, bl, idesc, 1u);
              mma2_tf32(tmem_d, ah, bh, idesc, 1u);
            }
            mma2_commit_both(&empty[s]);
          }
          if (ok) mma2_commit_both(&acc_full[buf]);
        }
      }
    }
  } else {
    asm volatile("setmaxnreg.inc.sync.aligned.u32 %0;" ::"n"(X3_REGS_HIGH));
    // ------------------------------------------------------------------ epilogue (warps 4..11, both CTAs)
    const int quad = warp & 3;
    const int half = (warp - 4) >> 2;
    const int row = quad * 32 + lane;
    int ci = 0;
    bool alive = true;
    for (int ti = 0; ti < my_tiles && alive; ++ti) {
      const int t = ti * p.P + pair;
      const int m0 = (t / p.tiles_n) * (2 * BM) + (int)rank * BM, n0 = (t % p.tiles_n) * bn;
      const int n_cc = min(bn / 32, (p.N - n0 + 31) / 32);       // column chunks of this tile that exist
      float run[4][32];                                          // this warp's chunks: half, half + 2, half + 4, half + 6
      for (int ch = 0; ch < n_chunks_k; ++ch, ++ci) {
        const int buf = ci & 1;
        const uint32_t aph = (ci >> 1) & 1;
        int good = 1;
        if (lane == 0) good = wait_or_abort(&acc_full[buf], aph, abort_flag, p.err, 3) ? 1 : 0;
        good = __shfl_sync(0xffffffffu, good, 0);
        if (!good) { alive = false; break; }
        tc_fence_after();
#pragma unroll
        for (int j = 0; j < 4; ++j) {
          const int c = half + 2 * j;
          if (c < n_cc) {                                        // warp-uniform
            float v[32];
            tmem_ld32(tmem_base + ((uint32_t)(quad * 32) << 16) + (uint32_t)(buf * BN_MAX + c * 32), v);
            // (a select, not a branch: two code paths over the 128 sums would double their registers)
#pragma unroll
            for (int i = 0; i < 32; ++i) run[j][i] = (ch == 0 ? 0.f : run[j][i]) + v[i];
          }
        }
        tc_fence_before();
        __syncwarp();
        if (lane == 0) mbar_arrive_cluster(map_to_cta(smem_u32(&acc_empty[buf]), 0));
      }
      if (!alive) break;
      const int m = m0 + row;
      if (m >= p.M) continue;
      const float* zrow = p.dsig ? p.dsig + (long long)((m / p.dsig_div) % p.dsig_rows) * p.ld_dsig : nullptr;
      const float* crow = p.cin ? p.cin + (long long)m * p.ld_cin : nullptr;
      float* drow = p.D + (long long)m * p.ldd;
      const int n_opt = (p.sigmoid ? 1 : 0) + (p.dsig ? 1 : 0) + (p.cin ? 1 : 0);
      const int xmode = n_opt == 0 ? 0 : n_opt > 1 ? 4 : p.sigmoid ? 1 : p.dsig ? 2 : 3;
#pragma unroll
      for (int j = 0; j < 4; ++j) {
        const int c = half + 2 * j;
        if (c >= n_cc) continue;
        const int nb = n0 + c * 32;
        if (p.vec_epi && nb + 32 <= p.N) {
          float* const hrow = p.Dhi ? p.Dhi + (long long)m * p.ld_parts + nb : nullptr;
          float* const lrow = p.Dhi ? p.Dlo + (long long)m * p.ld_parts + nb : nullptr;
          switch (xmode) {
            case 0: x3_store_chunk<0>(p, run[j], zrow ? zrow + nb : nullptr, crow ? crow + nb : nullptr, drow + nb, nb, hrow, lrow); break;
            case 1: x3_store_chunk<1>(p, run[j], zrow ? zrow + nb : nullptr, crow ? crow + nb : nullptr, drow + nb, nb, hrow, lrow); break;
            case 2: x3_store_chunk<2>(p, run[j], zrow ? zrow + nb : nullptr, crow ? crow + nb : nullptr, drow + nb, nb, hrow, lrow); break;
            case 3: x3_store_chunk<3>(p, run[j], zrow ? zrow + nb : nullptr, crow ? crow + nb : nullptr, drow + nb, nb, hrow, lrow); break;
            default: x3_store_chunk<4>(p, run[j], zrow ? zrow + nb : nullptr, crow ? crow + nb : nullptr, drow + nb, nb, hrow, lrow); break;
          }
        } else {
#pragma unroll
          for (int i = 0; i < 32; ++i) {
            const int n = nb + i;
            if (n < p.N) {
              float x = run[j][i] + (p.bias ? __ldg(p.bias + n) : 0.f);
              if (p.sigmoid) x = 1.f / (1.f + expf(-x));
              if (zrow) { const float z = __ldg(zrow + n); x *= z * (1.f - z); }
              x *= p.alpha;
              if (crow) x = fmaf(p.beta, __ldg(crow + n), x);
              drow[n] = x;
              if (p.Dhi) {
                const float h = round_tf32(x);
                p.Dhi[(long long)m * p.ld_parts + n] = h;
                p.Dlo[(long long)m * p.ld_parts + n] = round_tf32(x - h);
              }
            }
          }
        }
      }
    }
  }
  tc_fence_before();
  cluster_sync_all();
  if (warp == 2) {
    tc_fence_after();
    asm volatile("tcgen05.dealloc.cta_group::2.sync.aligned.b32 %0, %1;" ::"r"(tmem_base), "r"(512) : "memory");
  }
}

// One CTA waits on an mbarrier that nothing ever arrives on, with the same bounded-wait code the GEMM
// roles use but a caller-chosen limit; it must record its code and return.  Exercises the path from a
// timed-out device wait to GN_ETIMEOUT on the host without hanging anything.
__global__ void timeout_probe_kernel(int* err, unsigned long long limit_ns) {
  __shared__ uint64_t bar;
  if (threadIdx.x == 0) {
    mbar_init(&bar, 1);
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    const unsigned long long t0 = globaltimer();
    while (!mbar_test_wait(&bar, 0)) {
      if (globaltimer() - t0 > limit_ns) { atomicCAS(err, 0, 9); break; }
    }
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

// 3-D view of a row-major [K][MN] matrix (MN contiguous): (32 inner columns, K rows, MN/32 column chunks).
// One box (32, BK, chunks) lands in shared memory as `chunks` consecutive [BK][32] blocks.  The last
// chunk of a row may extend past MN (into the next row, or up to 124 bytes past the last row), so the
// operand must be followed by that much readable memory.
bool make_map_mn3d(CUtensorMap* m, const float* base, long long K, long long MN, long long ld, int chunks) {
  EncodeTiledFn fn = encode_fn();
  if (!fn) return false;
  cuuint64_t dims[3] = {32, (cuuint64_t)K, (cuuint64_t)((MN + 31) / 32)};
  cuuint64_t strides[2] = {(cuuint64_t)ld * 4, 128};
  cuuint32_t box[3] = {32, (cuuint32_t)BK, (cuuint32_t)chunks};
  cuuint32_t estr[3] = {1, 1, 1};
  CUresult r = fn(m, CU_TENSOR_MAP_DATA_TYPE_TFLOAT32, 3, const_cast<float*>(base), dims, strides, box, estr,
                  CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B_ATOM_32B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                  CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
  return r == CUDA_SUCCESS;
}

inline bool aligned16(const void* p) { return (reinterpret_cast<uintptr_t>(p) & 15) == 0; }

constexpr int kStages = 4;
constexpr int kSmemBytes = kStages * (A_STAGE_BYTES + BN_MAX * BK * 4) + 1024 + 256;

int num_sms() {
  static int n = 0;
  if (n == 0) {
    int dev = 0;
    cudaGetDevice(&dev);
    if (cudaDeviceGetAttribute(&n, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess || n <= 0) n = 148;
  }
  return n;
}

// Tile width against wave quantisation: every CTA runs ceil(tiles / SMs) tiles.  Measured tile times
// on B200 fit (320 + bn) units: the operand pipeline is latency-bound, so a narrower tile is only
// slightly cheaper and the width that minimises the number of waves usually wins.
int choose_bn(int M, int N) {
  const long long tiles_m = (M + BM - 1) / BM;
  const int sms = num_sms();
  int best = 256;
  long long best_cost = -1;
  for (int bn = 256; bn >= 128; bn -= 32) {
    const long long tiles = tiles_m * ((N + bn - 1) / bn);
    const long long cost = ((tiles + sms - 1) / sms) * (320 + bn);
    if (best_cost < 0 || cost < best_cost) { best_cost = cost; best = bn; }
  }
  if (N <= 64) best = 64;
  if (N <= 32) best = 32;
  return best;
}

}  // namespace

int launch_timeout_probe(int* err_flag, unsigned long long limit_ns, cudaStream_t st) {
  timeout_probe_kernel<<<1, 32, 0, st>>>(err_flag, limit_ns);
  return 1;
}

bool gemm_tf32_eligible(const GemmArgs& g) {
  if (g.M < 1 || g.N < 1) return false;
  if (!aligned16(g.A1) || !aligned16(g.B1) || g.lda1 % 4 || g.ldb1 % 4) return false;
  if (g.A2 && (!aligned16(g.A2) || !aligned16(g.B2) || g.lda2 % 4 || g.ldb2 % 4)) return false;
  if (!encode_fn()) return false;
  return true;
}

constexpr int kStages2 = 6;
constexpr int kMaxSlices = 16;   // K slices per left-over tile
constexpr int kSmemBytes2 = kStages2 * STAGE2_BYTES + 1024 + 256;

// Two-CTA tile width (a multiple of 64 so that each CTA's half is whole 32-column chunks).  With the
// work split evenly over the pairs (stream-K) only the padding of N to whole tiles costs anything;
// without it the number of waves decides as well.
int choose_bn2(int M, int N, bool stream_k, int fixed_cost = 320) {
  const long long tiles_m = (M + 2 * BM - 1) / (2 * BM);
  const int pairs = num_sms() / 2;
  int best = 256;
  long long best_cost = -1;
  for (int bn = 256; bn >= 128; bn -= 64) {
    const long long tiles_n = (N + bn - 1) / bn;
    const long long tiles = tiles_m * tiles_n;
    const long long cost = (stream_k ? tiles_n : (tiles + pairs - 1) / pairs) * (fixed_cost + bn);
    if (best_cost < 0 || cost < best_cost) { best_cost = cost; best = bn; }
  }
  return best;
}

int64_t gemm_tf32_workspace_floats() { return (int64_t)(num_sms() / 2) * 2 * BM * BN_MAX; }
int gemm_tf32_workspace_flags() { return num_sms() / 2; }

namespace {

// Launch with the programmatic stream-serialisation attribute (see grid_dep_wait above).
template <class... KArgs, class... Args>
cudaError_t launch_pdl(void (*kernel)(KArgs...), int grid, int block, int smem, cudaStream_t st, Args&&... args) {
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = dim3((unsigned)grid, 1, 1);
  cfg.blockDim = dim3((unsigned)block, 1, 1);
  cfg.dynamicSmemBytes = (size_t)smem;
  cfg.stream = st;
  cudaLaunchAttribute attr[1];
  attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  attr[0].val.programmaticStreamSerializationAllowed = 1;
  cfg.attrs = attr;
  cfg.numAttrs = 1;
  return cudaLaunchKernelEx(&cfg, kernel, std::forward<Args>(args)...);
}

// Tensor maps and kernel parameters of one problem for a given tile width (two_cta: 256 x bn tiles of a CTA pair).
bool setup_problem(const GemmArgs& g, bool two_cta, int bn, int* err_flag, CUtensorMap* maps, Tf32Params& p) {
  const int b_rows = two_cta ? bn / 2 : bn;      // B rows staged per CTA
  const float* As[2] = {g.A1, g.A2};
  const float* Bs[2] = {g.B1, g.B2};
  const int Ks[2] = {g.K1, g.A2 ? g.K2 : 0};
  const long long lda[2] = {g.lda1, g.lda2}, ldb[2] = {g.ldb1, g.ldb2};
  for (int s = 0; s < 2; ++s) {
    const int src = As[s] ? s : 0;  // unused second pair: repeat the first (never dereferenced)
    bool ok;
    const CUtensorMapSwizzle kmaj = CU_TENSOR_MAP_SWIZZLE_128B, mnmaj = CU_TENSOR_MAP_SWIZZLE_128B_ATOM_32B;
    if (g.a_kmajor)      ok = make_map(&maps[2 * s], As[src], g.M, Ks[src], lda[src], BK, BM, kmaj);
    else if (g.mn_padded) ok = make_map_mn3d(&maps[2 * s], As[src], Ks[src], g.M, lda[src], BM / 32);
    else                 ok = make_map(&maps[2 * s], As[src], Ks[src], g.M, lda[src], 32, BK, mnmaj);
    if (g.b_kmajor)      ok = ok && make_map(&maps[2 * s + 1], Bs[src], g.N, Ks[src], ldb[src], BK, b_rows, kmaj);
    else if (g.mn_padded) ok = ok && make_map_mn3d(&maps[2 * s + 1], Bs[src], Ks[src], g.N, ldb[src], b_rows / 32);
    else                 ok = ok && make_map(&maps[2 * s + 1], Bs[src], Ks[src], g.N, ldb[src], 32, BK, mnmaj);
    if (!ok) return false;
  }
  p = Tf32Params{};
  p.M = g.M; p.N = g.N;
  p.kblocks[0] = (Ks[0] + BK - 1) / BK;
  p.kblocks[1] = (Ks[1] + BK - 1) / BK;
  p.a_mn = g.a_kmajor ? 0 : 1; p.b_mn = g.b_kmajor ? 0 : 1;
  p.a_3d = (p.a_mn && g.mn_padded) ? 1 : 0; p.b_3d = (p.b_mn && g.mn_padded) ? 1 : 0;
  p.D = g.D; p.ldd = g.ldd;
  p.bias = g.bias; p.sigmoid = g.sigmoid;
  p.dsig = g.dsig; p.ld_dsig = g.ld_dsig; p.dsig_rows = g.dsig_rows > 0 ? g.dsig_rows : 1; p.dsig_div = g.dsig_div > 0 ? g.dsig_div : 1;
  p.alpha = g.alpha;
  p.cin = g.cin; p.ld_cin = g.ld_cin; p.beta = g.beta;
  p.vec_epi = aligned16(g.D) && (g.ldd % 4 == 0) && (!g.bias || aligned16(g.bias)) &&
              (!g.dsig || (aligned16(g.dsig) && g.ld_dsig % 4 == 0)) &&
              (!g.cin || (aligned16(g.cin) && g.ld_cin % 4 == 0));
  p.bn = bn;
  p.tiles_n = (g.N + bn - 1) / bn;
  p.tiles = ((g.M + (two_cta ? 2 : 1) * BM - 1) / ((two_cta ? 2 : 1) * BM)) * p.tiles_n;
  p.err = err_flag;
  p.slices = 1;
  return true;
}

void set_kernel_attributes() {
  static bool done = false;
  if (!done) {
    cudaFuncSetAttribute(gemm_tf32_kernel<kStages>, cudaFuncAttributeMaxDynamicSharedMemorySize, kSmemBytes);
    cudaFuncSetAttribute(gemm_tf32_2cta_kernel<kStages2>, cudaFuncAttributeMaxDynamicSharedMemorySize, kSmemBytes2);
    done = true;
  }
}

inline bool suits_pair_kernel(const GemmArgs& g) { return g.M > BM && g.N >= 128; }

}  // namespace

namespace {
// K slices for the tiles left over after the whole waves of a problem with `tiles` tiles of `total_kb` k-blocks on
// `pairs` CTA pairs (1 = whole tiles).  A sliced tile pays for a store and a re-read of its partial accumulators
// and for the wait between them, about as much as 25 to 30 k-blocks of main loop (measured: a 25-k-block tile is
// faster whole even when its wave is nearly empty, a 63-k-block tile gains from 2 slices on), so a tile is cut only
// if that saves more than this.
int choose_slices(int tiles, int total_kb, int pairs) {
  int rem = tiles % pairs;
  if (tiles < pairs) rem = tiles;
  if (rem == 0) return 1;
  int sl = pairs / rem;
  if (sl > kMaxSlices) sl = kMaxSlices;
  if (sl > total_kb) sl = total_kb;
  while (sl >= 2 && total_kb / sl < 4) --sl;
  if (sl < 2) return 1;
  return (double)total_kb * (1.0 - 1.0 / sl) >= 30.0 ? sl : 1;
}
}  // namespace

int launch_gemm_tf32(const GemmArgs& g, int* err_flag, float* sk_ws, int* sk_flags, cudaStream_t st) {
  set_kernel_attributes();
  const bool two_cta = g.two_cta >= 0 ? g.two_cta != 0 : suits_pair_kernel(g);
  bool stream_k = two_cta && sk_ws && sk_flags;
  const int pairs = num_sms() / 2;
  const int total_kb_all = (g.K1 + BK - 1) / BK + (g.A2 ? (g.K2 + BK - 1) / BK : 0);
  int bn = two_cta ? choose_bn2(g.M, g.N, stream_k) : choose_bn(g.M, g.N);
  if (stream_k) {
    // the width chosen for an even split of the work only stands if the left-over tiles will in fact be cut
    const int tiles = ((g.M + 2 * BM - 1) / (2 * BM)) * ((g.N + bn - 1) / bn);
    if (choose_slices(tiles, total_kb_all, pairs) < 2) { stream_k = false; bn = choose_bn2(g.M, g.N, false); }
  }
  if (two_cta) {
    GroupMaps gm;                              // (host copies; passed to the kernel by value)
    GroupParams gp = {};                       // (no dependencies, no signals)
    for (int k = 0; k < MAX_GROUP; ++k) gp.dep_prob[k] = -1;
    gp.n_prob = 1;
    Tf32Params& p = gp.pr[0];
    if (!setup_problem(g, true, bn, err_flag, gm.m[0], p)) return -1;
    const int total_kb = p.kblocks[0] + p.kblocks[1];
    p.sk_ws = sk_ws; p.sk_flags = sk_flags;
    p.P = p.tiles < pairs ? p.tiles : pairs;
    p.waves = p.tiles / p.P;
    p.rem = p.tiles - p.waves * p.P;
    int launch_pairs = p.P;
    if (stream_k) {
      const int sl = choose_slices(p.tiles, total_kb, pairs);
      if (sl >= 2) {
        if (p.tiles < pairs) { p.P = pairs; p.waves = 0; p.rem = p.tiles; }   // no full wave: every tile is cut
        p.slices = sl;
        if (p.waves == 0) launch_pairs = p.rem * p.slices;
      }
    }
    for (int q = 0; q <= MAX_PAIRS_LAUNCH; ++q) gp.rstart[0][q] = (unsigned short)(q < p.rem ? q : p.rem);
    launch_pdl(gemm_tf32_2cta_kernel<kStages2>, 2 * launch_pairs, 320, kSmemBytes2, st, gm, gp);
  } else {
    CUtensorMap maps[4];
    Tf32Params p;
    if (!setup_problem(g, false, bn, err_flag, maps, p)) return -1;
    const int grid = p.tiles < num_sms() ? p.tiles : num_sms();
    launch_pdl(gemm_tf32_kernel<kStages>, grid, 320, kSmemBytes, st, maps[0], maps[1], maps[2], maps[3], p);
  }
  return 1;
}

bool gemm_tf32_group_eligible(const GemmArgs* gs, int n) {
  if (n < 1 || n > MAX_GROUP || num_sms() / 2 > MAX_PAIRS_LAUNCH) return false;
  for (int i = 0; i < n; ++i)
    if (!gemm_tf32_eligible(gs[i]) || !suits_pair_kernel(gs[i]) || gs[i].two_cta == 0) return false;
  return true;
}

namespace {

// Tiles of problem slot k of a group (cost `cost` each) dealt to the P pairs on top of the loads they carry
// already: as many whole waves (tiles q, q + P, ... for every pair q) as every pair takes anyway, the rest as
// contiguous runs of the left-over tiles, so that the loads come out as even as whole tiles allow.
void deal_tiles(GroupParams& gp, int k, double cost, int P, double* load) {
  Tf32Params& p = gp.pr[k];
  p.P = P;
  int cnt[MAX_PAIRS_LAUNCH];
  // lowest level L with sum_q floor((L - load_q) / cost) >= tiles, by bisection on L
  double lo = 0.0, hi = 0.0;
  for (int q = 0; q < P; ++q) if (load[q] > hi) hi = load[q];
  hi += cost * (p.tiles / P + 2);
  for (int iter = 0; iter < 60; ++iter) {
    const double mid = 0.5 * (lo + hi);
    long long have = 0;
    for (int q = 0; q < P; ++q) if (mid > load[q]) have += (long long)((mid - load[q]) / cost);
    if (have >= p.tiles) hi = mid; else lo = mid;
  }
  long long have = 0;
  for (int q = 0; q < P; ++q) { cnt[q] = hi > load[q] ? (int)((hi - load[q]) / cost) : 0; have += cnt[q]; }
  // more than needed (several pairs cross a multiple of `cost` at the same level): take back from the fullest
  while (have > p.tiles) {
    int worst = -1;
    for (int q = 0; q < P; ++q)
      if (cnt[q] > 0 && (worst < 0 || load[q] + cnt[q] * cost > load[worst] + cnt[worst] * cost)) worst = q;
    --cnt[worst]; --have;
  }
  while (have < p.tiles) {                    // (rounding in the bisection)
    int best = 0;
    for (int q = 1; q < P; ++q)
      if (load[q] + cnt[q] * cost < load[best] + cnt[best] * cost) best = q;
    ++cnt[best]; ++have;
  }
  int waves = cnt[0];
  for (int q = 1; q < P; ++q) if (cnt[q] < waves) waves = cnt[q];
  p.waves = waves;
  p.rem = p.tiles - waves * P;
  int run = 0;
  for (int q = 0; q < P; ++q) { gp.rstart[k][q] = (unsigned short)run; run += cnt[q] - waves; load[q] += cnt[q] * cost; }
  for (int q = P; q <= MAX_PAIRS_LAUNCH; ++q) gp.rstart[k][q] = (unsigned short)run;
}

// time of one tile in k-blocks of a 256-wide tile: operand bytes per k-block (the feed bounds the main loop) plus a fixed part
double tile_cost(const Tf32Params& p) { return (p.kblocks[0] + p.kblocks[1]) * (256.0 + p.bn) / 512.0 + 8.0; }

}  // namespace

// Several problems in one launch of the CTA-pair kernel.
//   Independent problems (dep_prob == nullptr): taken longest tile first, the pairs' loads evened out on the host,
//   so the short tiles of one problem fill the partial last wave of another.
//   A chain (dep_prob[i] = index of the earlier problem whose output problem i reads, or -1; dep_all[i] != 0 if it
//   needs all of that output rather than the 256-row panel of its own tile): kept in the given order, every pair
//   works through the problems one after the other, and the head of a problem overlaps the tail of the one before.
//   `done` is a zeroed-by-this-call array of n * done_stride ints, done_stride > the number of 256-row panels.
int launch_gemm_tf32_group(const GemmArgs* gs, int n, const int* dep_prob, const int* dep_all, int* done,
                           int done_stride, int* err_flag, cudaStream_t st) {
  if (!gemm_tf32_group_eligible(gs, n)) return -1;
  set_kernel_attributes();
  GroupMaps gm;
  GroupParams gp = {};
  const int pairs = num_sms() / 2;
  struct Item { int src; double cost; };
  Item order[MAX_GROUP];
  Tf32Params tmp[MAX_GROUP];
  CUtensorMap tmaps[MAX_GROUP][4];
  long long total_tiles = 0;
  for (int i = 0; i < n; ++i) {
    const int bn = choose_bn2(gs[i].M, gs[i].N, true);
    if (!setup_problem(gs[i], true, bn, err_flag, tmaps[i], tmp[i])) return -1;
    if (tmp[i].tiles > 60000) return -1;       // (left-over tile indices are 16-bit)
    order[i].src = i;
    order[i].cost = tile_cost(tmp[i]);
    total_tiles += tmp[i].tiles;
  }
  const bool chain = dep_prob != nullptr;
  if (chain) {
    if (!done) return -1;
    for (int i = 0; i < n; ++i) {
      if (dep_prob[i] >= i) return -1;
      if (dep_prob[i] >= 0 && !dep_all[i] && gs[dep_prob[i]].M != gs[i].M) return -1;   // panels must coincide
      if ((gs[i].M + 2 * BM - 1) / (2 * BM) + 1 > done_stride) return -1;
    }
  } else {
    for (int i = 1; i < n; ++i)                 // insertion sort, longest tile first (stable)
      for (int j = i; j > 0 && order[j].cost > order[j - 1].cost; --j) { Item t = order[j]; order[j] = order[j - 1]; order[j - 1] = t; }
  }
  const int P = total_tiles < pairs ? (int)total_tiles : pairs;
  double load[MAX_PAIRS_LAUNCH];
  for (int q = 0; q < P; ++q) load[q] = 0.0;
  gp.n_prob = n;
  gp.done = done; gp.done_stride = done_stride;
  for (int k = 0; k < MAX_GROUP; ++k) { gp.dep_prob[k] = -1; gp.dep_all[k] = 0; gp.signal[k] = 0; }
  for (int k = 0; k < n; ++k) {
    const int i = order[k].src;
    gp.pr[k] = tmp[i];
    for (int j = 0; j < 4; ++j) gm.m[k][j] = tmaps[i][j];
    deal_tiles(gp, k, order[k].cost, P, load);
    if (chain && dep_prob[i] >= 0) {            // (a chain keeps its order: slot == index)
      gp.dep_prob[k] = dep_prob[i];
      gp.dep_all[k] = dep_all[i] ? 1 : 0;
      gp.signal[dep_prob[i]] |= dep_all[i] ? 2 : 1;
    }
  }
  if (chain && cudaMemsetAsync(done, 0, sizeof(int) * (size_t)n * done_stride, st) != cudaSuccess) return -1;
  launch_pdl(gemm_tf32_2cta_kernel<kStages2>, 2 * P, 320, kSmemBytes2, st, gm, gp);
  return 1;
}

// Host-only view of the work list a grouped launch would use (no device needed): for problems of the given shapes
// on `pairs` CTA pairs, counts[k * pairs + q] = tiles of the k-th problem IN LAUNCH ORDER that pair q runs,
// waves[k] = how many of them are whole waves (tiles q, q + pairs, ...), order[k] = index of that problem in the
// caller's list, tiles[k] = its tile count.  keep_order != 0 keeps the caller's order (a chain).  Returns the number
// of pairs the launch would use, or -1 for bad arguments.
namespace {
int plan_group_impl(int n, const int* M, const int* N, const int* K, int pairs, int keep_order, int* counts,
                    int* waves, int* order_out, int* tiles_out, double* makespan) {
  if (n < 1 || n > MAX_GROUP || pairs < 1 || pairs > MAX_PAIRS_LAUNCH) return -1;
  GroupParams gp = {};
  struct Item { int src; double cost; };
  Item order[MAX_GROUP];
  Tf32Params tmp[MAX_GROUP];
  long long total_tiles = 0;
  for (int i = 0; i < n; ++i) {
    if (M[i] < 1 || N[i] < 1 || K[i] < 1) return -1;
    const int bn = choose_bn2(M[i], N[i], true);
    tmp[i] = Tf32Params{};
    tmp[i].bn = bn;
    tmp[i].kblocks[0] = (K[i] + BK - 1) / BK;
    tmp[i].tiles_n = (N[i] + bn - 1) / bn;
    tmp[i].tiles = ((M[i] + 2 * BM - 1) / (2 * BM)) * tmp[i].tiles_n;
    order[i].src = i;
    order[i].cost = tile_cost(tmp[i]);
    total_tiles += tmp[i].tiles;
  }
  if (!keep_order)
    for (int i = 1; i < n; ++i)
      for (int j = i; j > 0 && order[j].cost > order[j - 1].cost; --j) { Item t = order[j]; order[j] = order[j - 1]; order[j - 1] = t; }
  const int P = total_tiles < pairs ? (int)total_tiles : pairs;
  double load[MAX_PAIRS_LAUNCH];
  for (int q = 0; q < P; ++q) load[q] = 0.0;
  for (int k = 0; k < n; ++k) {
    gp.pr[k] = tmp[order[k].src];
    deal_tiles(gp, k, order[k].cost, P, load);
    if (waves) waves[k] = gp.pr[k].waves;
    if (order_out) order_out[k] = order[k].src;
    if (tiles_out) tiles_out[k] = gp.pr[k].tiles;
    if (counts)
      for (int q = 0; q < pairs; ++q)
        counts[k * pairs + q] = q < P ? gp.pr[k].waves + (gp.rstart[k][q + 1] - gp.rstart[k][q]) : 0;
  }
  if (makespan) {
    *makespan = 0.0;
    for (int q = 0; q < P; ++q) if (load[q] > *makespan) *makespan = load[q];
  }
  return P;
}
}  // namespace

int gemm_tf32_plan_group(int n, const int* M, const int* N, const int* K, int pairs, int keep_order, int* counts,
                         int* waves, int* order_out, int* tiles_out) {
  return plan_group_impl(n, M, N, K, pairs, keep_order, counts, waves, order_out, tiles_out, nullptr);
}

// Load of the fullest CTA pair, in k-blocks of a 256-wide tile, if the problems went out as one grouped
// (keep_order == 0) or chained launch on this device; negative for bad arguments.  Host arithmetic only.
double gemm_tf32_group_makespan(int n, const int* M, const int* N, const int* K, int keep_order) {
  double ms = 0.0;
  if (plan_group_impl(n, M, N, K, num_sms() / 2, keep_order, nullptr, nullptr, nullptr, nullptr, &ms) < 0) return -1.0;
  return ms;
}

// ---- error-compensated form ---------------------------------------------------------------------
// 4 k-blocks = 128 terms (384 products) per accumulation in tensor memory: the truncation bias of one chunk stays
// below 1e-6 relative (measured), and the running sums outside are round-to-nearest.
constexpr int kChunkKb = 4;
constexpr int kSmemBytes3 = X3_STAGES * X3_STAGE_BYTES + 1024 + 256;

// The register split of the kernel (128 x 56 + 256 x 224) must not exceed what the block is launched with, and
// the kernel needs its dynamic shared memory granted: checked once.
bool gemm_tf32x3_usable() {
  static int usable = -1;
  if (usable < 0) {
    cudaFuncAttributes fa;
    usable = encode_fn() != nullptr &&
             cudaFuncGetAttributes(&fa, gemm_tf32x3_kernel<X3_STAGES>) == cudaSuccess &&
             fa.numRegs * X3_THREADS >= 128 * X3_REGS_LOW + 256 * X3_REGS_HIGH &&
             cudaFuncSetAttribute(gemm_tf32x3_kernel<X3_STAGES>, cudaFuncAttributeMaxDynamicSharedMemorySize, kSmemBytes3) == cudaSuccess;
    cudaGetLastError();
  }
  return usable != 0;
}

bool gemm_tf32x3_eligible(const GemmArgs& g) {
  // the operands' own alignment does not matter: the kernel reads their hi / lo copies
  return g.M > BM && g.N >= 128 && gemm_tf32x3_usable();
}

int launch_gemm_tf32x3(const GemmArgs& g, int* err_flag, cudaStream_t st) {
  const bool usable = gemm_tf32x3_usable();
  if (!usable || !g.A1lo || !g.B1lo || (g.A2 && (!g.A2lo || !g.B2lo))) return -1;
  // this kernel is bound by its MMAs, not by the operand feed: a tile's time is nearly proportional to its width
  // (measured: 96 + bn units against the TF32 kernel's 320 + bn), so narrower tiles win more often
  const int bn = choose_bn2(g.M, g.N, false, 96);
  const int b_rows = bn / 2;
  const float* Ah[2] = {g.A1, g.A2}; const float* Al[2] = {g.A1lo, g.A2lo};
  const float* Bh[2] = {g.B1, g.B2}; const float* Bl[2] = {g.B1lo, g.B2lo};
  const int Ks[2] = {g.K1, g.A2 ? g.K2 : 0};
  const long long lda[2] = {g.lda1, g.lda2}, ldb[2] = {g.ldb1, g.ldb2};
  MapSet maps;
  const CUtensorMapSwizzle kmaj = CU_TENSOR_MAP_SWIZZLE_128B;
  for (int s = 0; s < MAX_PAIRS; ++s) {
    const int src = Ah[s] ? s : 0;      // unused second pair: repeat the first (never dereferenced)
    bool ok = true;
    const float* as[2] = {Ah[src], Al[src]}; CUtensorMap* am[2] = {&maps.a_hi[s], &maps.a_lo[s]};
    const float* bs[2] = {Bh[src], Bl[src]}; CUtensorMap* bm[2] = {&maps.b_hi[s], &maps.b_lo[s]};
    for (int h = 0; h < 2 && ok; ++h) {
      if (g.a_kmajor) ok = make_map(am[h], as[h], g.M, Ks[src], lda[src], BK, BM, kmaj);
      else            ok = make_map_mn3d(am[h], as[h], Ks[src], g.M, lda[src], BM / 32);
      if (g.b_kmajor) ok = ok && make_map(bm[h], bs[h], g.N, Ks[src], ldb[src], BK, b_rows, kmaj);
      else            ok = ok && make_map_mn3d(bm[h], bs[h], Ks[src], g.N, ldb[src], b_rows / 32);
    }
    if (!ok) return -1;
  }
  Tf32Params p{};
  X3Params xp{};
  p.M = g.M; p.N = g.N;
  xp.n_pairs = g.A2 ? 2 : 1;
  for (int s = 0; s < xp.n_pairs; ++s) xp.kblocks[s] = (Ks[s] + BK - 1) / BK;
  xp.chunk_kb = kChunkKb;
  p.a_mn = g.a_kmajor ? 0 : 1; p.b_mn = g.b_kmajor ? 0 : 1;
  p.a_3d = p.a_mn; p.b_3d = p.b_mn;
  p.D = g.D; p.ldd = g.ldd;
  p.bias = g.bias; p.sigmoid = g.sigmoid;
  p.dsig = g.dsig; p.ld_dsig = g.ld_dsig; p.dsig_rows = g.dsig_rows > 0 ? g.dsig_rows : 1; p.dsig_div = g.dsig_div > 0 ? g.dsig_div : 1;
  p.alpha = g.alpha;
  p.cin = g.cin; p.ld_cin = g.ld_cin; p.beta = g.beta;
  p.vec_epi = aligned16(g.D) && (g.ldd % 4 == 0) && (!g.bias || aligned16(g.bias)) &&
              (!g.dsig || (aligned16(g.dsig) && g.ld_dsig % 4 == 0)) &&
              (!g.cin || (aligned16(g.cin) && g.ld_cin % 4 == 0));
  p.Dhi = g.Dhi; p.Dlo = g.Dlo; p.ld_parts = g.ld_parts;
  if (p.Dhi && !(aligned16(g.Dhi) && aligned16(g.Dlo) && g.ld_parts % 4 == 0)) return -1;
  p.bn = bn;
  p.tiles_n = (g.N + bn - 1) / bn;
  p.err = err_flag;
  p.tiles = ((g.M + 2 * BM - 1) / (2 * BM)) * p.tiles_n;
  const int pairs = num_sms() / 2;
  p.P = p.tiles < pairs ? p.tiles : pairs;
  p.waves = p.tiles / p.P;
  p.rem = p.tiles - p.waves * p.P;
  p.slices = 1;
  launch_pdl(gemm_tf32x3_kernel<X3_STAGES>, 2 * p.P, X3_THREADS, kSmemBytes3, st, maps, p, xp);
  return 1;
}

}  // namespace gn
