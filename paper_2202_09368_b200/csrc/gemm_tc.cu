// Batched bf16 GEMM on the 5th-generation tensor cores (tcgen05) for the expert FFNs (Eq. 3),
// their backward contractions, and the gate of Eq. 2 (with the row softmax in the epilogue).
//
//   C[b] (M x N, fp32 accumulate) = A[b] (M x K) . B[b] (K x N),  b = 0 .. batches-1
//
// One persistent CTA per SM, 320 threads, warp-specialised:
//   warp 0      TMA producer: fills a ring of shared-memory stages (A 128 x 64, B BN x 64 bf16,
//               128-byte swizzle) with cp.async.bulk.tensor, one mbarrier per stage;
//   warp 1      MMA issuer: one thread issues tcgen05.mma (M = 128, N = BN, K = 16) on shared-memory
//               descriptors, accumulating in tensor memory; tcgen05.commit releases stages and
//               publishes finished accumulators.  Two accumulators (2 x BN columns) are kept so the
//               epilogue of one tile overlaps the main loop of the next;
//   warps 2..9  epilogue (two per 32-lane quarter of tensor memory, half the columns each): tcgen05.ld
//               the accumulator (one row of the tile per thread), apply the fused function (GeLU,
//               GeLU', slot-row sum, softmax), stage the result in shared memory and hand it to TMA stores.
// Split-K mode (k_split): the batch index selects a cut of the K axis of one product and the partial
// results are fp32 (dWg = X^T . dL over the tokens).
// Operands may be K-major (K contiguous in memory) or MN-major (M or N contiguous); the weights
// W1, W2 [E, d, d'] and the activations are never transposed in memory, the shared-memory
// descriptors carry the orientation.  Three-dimensional tensor maps (inner, rows, batch) let the
// TMA unit zero-fill whatever a tile overhangs, so ragged M, N and K need no special code.
// Tiles are ordered with M fastest so that CTAs running together share the same weight tile in L2
// (with N fastest for the weight gradients, whose output dominates: see launch_gemm_tc).
//
// Two-CTA mode (CTAS = 2, used whenever M > 128): the two CTAs of a cluster work on one
// 256 x BN tile.  Each loads its own 128 rows of A and its own half (BN / 2 rows) of B, so a
// k-block costs each SM 32 KiB of fill instead of 48 KiB for the same 128 x 256 block of
// accumulators; the main loop is bound by the L2 -> shared-memory fill rate, which is what
// this buys.  Both producers announce their bytes on, and their copies complete on, the
// full barrier of the even ("leader") CTA; the leader's thread issues tcgen05.mma.cta_group::2,
// which reads both CTAs' shared memory and writes both CTAs' tensor memory (each keeps its own
// 128 rows); tcgen05.commit with a two-CTA multicast releases the stage and publishes the
// accumulator in both.  Each CTA's epilogue warps drain their own rows and report to the
// leader's barrier.  Loads never use cluster multicast.
// A pair takes 256 x 512 tiles (BN = 512) when the contraction is long and the epilogue only converts and
// stores (GEMM-2, dX_in): two MMAs per K step share the A operand, a k-block costs each SM 48 KiB for twice
// the accumulators (a quarter less fill per flop, which under a power cap is what the clocks follow), and
// the one accumulator fills tensor memory, so the epilogue is not overlapped: 4 to 8 store chunks per warp
// against a main loop of at least 256 MMAs.  The epilogues that evaluate GeLU or GeLU' are bound by
// their arithmetic and stay on 256-column tiles, where the next tile's main loop hides them.
//
// Every wait on an mbarrier is bounded: after about two seconds the kernel records
// EC_ERR_TIMEOUT in the status word, all roles leave their loops and the CTA exits in order.
#include "internal.h"

#include <cuda.h>
#include <cudaTypedefs.h>
#include <atomic>
#include <mutex>
#include <type_traits>
#include <string.h>

namespace ecmoe {

namespace {

constexpr int BM = 128, BK = 64, UK = 16;
constexpr int kEpiWarps = 8;                         // two per TMEM lane quarter, each takes half the columns
constexpr int kThreads = 32 * (2 + kEpiWarps);
constexpr int kABytes = BM * BK * 2;                 // 16 KiB
constexpr int kSmemBudget = 224 * 1024;              // operand stages plus the epilogue's staging
constexpr int kStagingPerWarp = 8192;                // two 4 KiB buffers of 32 rows x 128 bytes
constexpr int EPI_STORE_F32 = 5;                     // like EPI_STORE with fp32 output
constexpr unsigned long long kWaitNs = 2000000000ull;
constexpr int kWideMinK = 2048;                      // contraction length from which a CTA pair takes 256 x 512 tiles

// bn = rows of B one CTA loads per k-block (BN / CTAS)
__host__ __device__ constexpr int stage_bytes(int bn) { return kABytes + bn * BK * 2; }
// Staging for the epilogue: every warp's when the tile is split between the warp pairs, else (a 64-wide tile with
// the softmax, drained by the first four warps alone) only theirs, which leaves room for more stages.
__host__ __device__ constexpr int staging_bytes(int bn_tile, int epi) { return (epi == EPI_SOFTMAX && bn_tile < 128 ? 4 : kEpiWarps) * kStagingPerWarp; }
__host__ __device__ constexpr int num_stages(int bn, int staging) {
  return (kSmemBudget - staging) / stage_bytes(bn) > 8 ? 8 : (kSmemBudget - staging) / stage_bytes(bn);
}
// Two accumulators of BN columns (a power of two for BN = 64, 128, 256), or one of 512.  A CTA pair takes all 512
// columns, so both CTAs are certain to get base address 0: one tcgen05.mma writes the same
// tensor-memory address in both.
__host__ __device__ constexpr int tmem_cols(int bn, int ctas) { return ctas == 2 ? 512 : (2 * bn < 32 ? 32 : 2 * bn); }

struct TcParams {
  int M, N, K, batches;
  int a_mn, b_mn;
  int tiles_m, tiles_n, total_tiles, kblocks;
  int n_fast;                                        // consecutive tiles run along N (else along M)
  int gelu;
  const bf16* Zin;                                   // EPI_GELU_GRAD reads Z directly; every output leaves through a tensor map
  int64_t ldc, batch_c;
  int* status;
  int k_split;                                       // batches are cuts of one product along K
  int skip_c;                                        // EPI_GELU: only H = GeLU(acc) is stored, the accumulator itself is not
  const int32_t* row_ptr; const int32_t* slots; const bf16* rows; int64_t ld_rows;   // EPI_ADD_SLOTS
  int64_t slots_total;                               // rows of `rows`: what the debug build checks the slot ids against
  const int32_t* batch_rows; int ragged;             // meaningful rows per batch along M (1) or K (2), zeros beyond
  const bf16* bias;                                  // EPI_GELU, EPI_STORE_F32: bias[b * N + n] joins every row of the accumulator
  const int32_t* a_rows; int64_t a_rows_batch; int a_rows_total;   // A's stored rows come from one matrix through this index list (tmA is then 2-D)
};

// ---------------------------------------------------------------------------------------------
// PTX wrappers
// ---------------------------------------------------------------------------------------------
__device__ __forceinline__ uint32_t smem_u32(const void* p) { return (uint32_t)__cvta_generic_to_shared(p); }
__device__ __forceinline__ unsigned long long globaltimer() {
  unsigned long long t; asm volatile("mov.u64 %0, %%globaltimer;" : "=l"(t)); return t;
}
__device__ __forceinline__ void mbar_init(uint32_t bar, uint32_t count) {
  asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(bar), "r"(count));
}
__device__ __forceinline__ void mbar_expect_tx(uint32_t bar, uint32_t bytes) {
  asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(bar), "r"(bytes) : "memory");
}
__device__ __forceinline__ void mbar_arrive(uint32_t bar) {
  asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(bar) : "memory");
}
__device__ __forceinline__ bool mbar_try(uint32_t bar, uint32_t parity) {
  uint32_t ok;
  asm volatile("{\n .reg .pred p;\n mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n selp.u32 %0, 1, 0, p;\n}\n"
               : "=r"(ok) : "r"(bar), "r"(parity) : "memory");
  return ok != 0;
}
// Bounded wait.  Returns false when the limit expired or another role already gave up.
__device__ __forceinline__ bool mbar_wait(uint32_t bar, uint32_t parity, volatile int* abort_flag, int* status, int where) {
  if (mbar_try(bar, parity)) return true;
  const unsigned long long t0 = globaltimer();
  for (uint32_t spin = 1;; ++spin) {
    if (mbar_try(bar, parity)) return true;
    if ((spin & 63u) == 0) {
      if (*abort_flag) return false;
      if (globaltimer() - t0 > kWaitNs) {
        *abort_flag = 1;
        atomicExch(status + 1, where);
        atomicExch(status, 5 /* EC_ERR_TIMEOUT */);
        return false;
      }
    }
  }
}
__device__ __forceinline__ void tma_load_3d(uint32_t dst, const CUtensorMap* tm, uint32_t bar, int c0, int c1, int c2) {
  asm volatile("cp.async.bulk.tensor.3d.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%3, %4, %5}], [%2];"
               ::"r"(dst), "l"(tm), "r"(bar), "r"(c0), "r"(c1), "r"(c2) : "memory");
}
// Two-CTA forms.  The barrier operands are shared::cluster addresses (possibly the peer's).
__device__ __forceinline__ uint32_t cluster_ctarank() { uint32_t r; asm volatile("mov.u32 %0, %%cluster_ctarank;" : "=r"(r)); return r; }
__device__ __forceinline__ uint32_t map_to_cta(uint32_t saddr, uint32_t rank) {
  uint32_t r; asm volatile("mapa.shared::cluster.u32 %0, %1, %2;" : "=r"(r) : "r"(saddr), "r"(rank)); return r;
}
__device__ __forceinline__ void mbar_arrive_cluster(uint32_t bar) {
  asm volatile("mbarrier.arrive.release.cluster.shared::cluster.b64 _, [%0];" ::"r"(bar) : "memory");
}
__device__ __forceinline__ void tma_load_3d_pair(uint32_t dst, const CUtensorMap* tm, uint32_t bar, int c0, int c1, int c2) {
  asm volatile("cp.async.bulk.tensor.3d.cta_group::2.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%3, %4, %5}], [%2];"
               ::"r"(dst), "l"(tm), "r"(bar), "r"(c0), "r"(c1), "r"(c2) : "memory");
}
// Named barriers over the four epilogue warps that share a half of the tile's columns (ids 1 and 2; 0 is __syncthreads).
__device__ __forceinline__ void half_sync(int half) { asm volatile("bar.sync %0, 128;" ::"r"(1 + half) : "memory"); }
__device__ __forceinline__ bool half_all(int half, bool ok) {          // true when `ok` holds in all 128 threads
  uint32_t r;
  asm volatile("{\n .reg .pred p, q;\n setp.ne.b32 p, %2, 0;\n barrier.cta.red.and.pred q, %1, 128, p;\n selp.u32 %0, 1, 0, q;\n}\n"
               : "=r"(r) : "r"(1 + half), "r"((uint32_t)ok) : "memory");
  return r != 0;
}
// Row-indexed loads (tile::gather4): four rows of a 2-D tensor, chosen by index, 64 elements (128 bytes) of each
// starting at column c0, land as four consecutive 128-byte rows at dst.  The tensor map's box is one row high.
__device__ __forceinline__ void tma_gather4(uint32_t dst, const CUtensorMap* tm, uint32_t bar, int c0, int r0, int r1, int r2, int r3) {
  asm volatile("cp.async.bulk.tensor.2d.shared::cluster.global.tile::gather4.mbarrier::complete_tx::bytes [%0], [%1, {%3, %4, %5, %6, %7}], [%2];"
               ::"r"(dst), "l"(tm), "r"(bar), "r"(c0), "r"(r0), "r"(r1), "r"(r2), "r"(r3) : "memory");
}
__device__ __forceinline__ void tma_gather4_pair(uint32_t dst, const CUtensorMap* tm, uint32_t bar, int c0, int r0, int r1, int r2, int r3) {
  asm volatile("cp.async.bulk.tensor.2d.cta_group::2.shared::cluster.global.tile::gather4.mbarrier::complete_tx::bytes [%0], [%1, {%3, %4, %5, %6, %7}], [%2];"
               ::"r"(dst), "l"(tm), "r"(bar), "r"(c0), "r"(r0), "r"(r1), "r"(r2), "r"(r3) : "memory");
}
__device__ __forceinline__ void cluster_sync_all() {
  asm volatile("barrier.cluster.arrive.release.aligned;\n barrier.cluster.wait.acquire.aligned;" ::: "memory");
}
__device__ __forceinline__ void tc_commit_pair(uint32_t bar) {   // arrives on the barrier at this offset in both CTAs
  asm volatile("tcgen05.commit.cta_group::2.mbarrier::arrive::one.shared::cluster.multicast::cluster.b64 [%0], %1;"
               ::"r"(bar), "h"((uint16_t)3) : "memory");
}
__device__ __forceinline__ void tc_mma_pair(uint32_t d_tmem, uint64_t adesc, uint64_t bdesc, uint32_t idesc, uint32_t accumulate) {
  asm volatile("{\n .reg .pred p;\n setp.ne.b32 p, %4, 0;\n tcgen05.mma.cta_group::2.kind::f16 [%0], %1, %2, %3, p;\n}\n"
               ::"r"(d_tmem), "l"(adesc), "l"(bdesc), "r"(idesc), "r"(accumulate) : "memory");
}
__device__ __forceinline__ void tma_store_3d(const CUtensorMap* tm, uint32_t src, int c0, int c1, int c2) {
  asm volatile("cp.async.bulk.tensor.3d.global.shared::cta.bulk_group [%0, {%2, %3, %4}], [%1];"
               ::"l"(tm), "r"(src), "r"(c0), "r"(c1), "r"(c2) : "memory");
}
__device__ __forceinline__ void bulk_commit() { asm volatile("cp.async.bulk.commit_group;" ::: "memory"); }
template <int N> __device__ __forceinline__ void bulk_wait_read() { asm volatile("cp.async.bulk.wait_group.read %0;" ::"n"(N) : "memory"); }
__device__ __forceinline__ void bulk_wait_all() { asm volatile("cp.async.bulk.wait_group 0;" ::: "memory"); }
__device__ __forceinline__ void fence_async_smem() { asm volatile("fence.proxy.async.shared::cta;" ::: "memory"); }
__device__ __forceinline__ void tc_fence_before() { asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void tc_fence_after() { asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void tc_commit(uint32_t bar) {
  asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(bar) : "memory");
}
__device__ __forceinline__ void tc_mma(uint32_t d_tmem, uint64_t adesc, uint64_t bdesc, uint32_t idesc, uint32_t accumulate) {
  asm volatile("{\n .reg .pred p;\n setp.ne.b32 p, %4, 0;\n tcgen05.mma.cta_group::1.kind::f16 [%0], %1, %2, %3, p;\n}\n"
               ::"r"(d_tmem), "l"(adesc), "l"(bdesc), "r"(idesc), "r"(accumulate) : "memory");
}
__device__ __forceinline__ void tc_ld32(uint32_t taddr, uint32_t* r) {
  asm volatile(
      "tcgen05.ld.sync.aligned.32x32b.x32.b32 "
      "{%0, %1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15, "
      "%16, %17, %18, %19, %20, %21, %22, %23, %24, %25, %26, %27, %28, %29, %30, %31}, [%32];"
      : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7]),
        "=r"(r[8]), "=r"(r[9]), "=r"(r[10]), "=r"(r[11]), "=r"(r[12]), "=r"(r[13]), "=r"(r[14]), "=r"(r[15]),
        "=r"(r[16]), "=r"(r[17]), "=r"(r[18]), "=r"(r[19]), "=r"(r[20]), "=r"(r[21]), "=r"(r[22]), "=r"(r[23]),
        "=r"(r[24]), "=r"(r[25]), "=r"(r[26]), "=r"(r[27]), "=r"(r[28]), "=r"(r[29]), "=r"(r[30]), "=r"(r[31])
      : "r"(taddr) : "memory");
  asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory");
}

// The same load without the wait, so that several can be in flight; tc_ld_wait() completes them all.
__device__ __forceinline__ void tc_ld32_issue(uint32_t taddr, uint32_t* r) {
  asm volatile(
      "tcgen05.ld.sync.aligned.32x32b.x32.b32 "
      "{%0, %1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15, "
      "%16, %17, %18, %19, %20, %21, %22, %23, %24, %25, %26, %27, %28, %29, %30, %31}, [%32];"
      : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7]),
        "=r"(r[8]), "=r"(r[9]), "=r"(r[10]), "=r"(r[11]), "=r"(r[12]), "=r"(r[13]), "=r"(r[14]), "=r"(r[15]),
        "=r"(r[16]), "=r"(r[17]), "=r"(r[18]), "=r"(r[19]), "=r"(r[20]), "=r"(r[21]), "=r"(r[22]), "=r"(r[23]),
        "=r"(r[24]), "=r"(r[25]), "=r"(r[26]), "=r"(r[27]), "=r"(r[28]), "=r"(r[29]), "=r"(r[30]), "=r"(r[31])
      : "r"(taddr) : "memory");
}
__device__ __forceinline__ void tc_ld_wait() { asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory"); }

// Shared-memory matrix descriptor, 128-byte swizzle.  lbo / sbo in bytes.
__device__ __forceinline__ uint64_t make_desc(uint32_t saddr, uint32_t lbo, uint32_t sbo) {
  return (uint64_t)((saddr & 0x3FFFFu) >> 4) | ((uint64_t)(lbo >> 4) << 16) | ((uint64_t)(sbo >> 4) << 32) |
         (1ull << 46) | (2ull << 61);
}

// Packed fp32 pairs: two lanes of arithmetic per instruction (fma.rn.f32x2 and friends).
__device__ __forceinline__ unsigned long long pk2(float a, float b) {
  return (unsigned long long)__float_as_uint(a) | ((unsigned long long)__float_as_uint(b) << 32);
}
__device__ __forceinline__ unsigned long long fma2(unsigned long long a, unsigned long long b, unsigned long long c) {
  unsigned long long d; asm("fma.rn.f32x2 %0, %1, %2, %3;" : "=l"(d) : "l"(a), "l"(b), "l"(c)); return d;
}
__device__ __forceinline__ unsigned long long mul2(unsigned long long a, unsigned long long b) {
  unsigned long long d; asm("mul.rn.f32x2 %0, %1, %2;" : "=l"(d) : "l"(a), "l"(b)); return d;
}
__device__ __forceinline__ float lo2(unsigned long long v) { return __uint_as_float((unsigned)v); }
__device__ __forceinline__ float hi2(unsigned long long v) { return __uint_as_float((unsigned)(v >> 32)); }

// Phi(z) = (1 + erf(z / sqrt 2)) / 2 for two values at once, without special-function instructions:
// erf(u) = u Q(t) with t = 2 u^2 / U^2 - 1 in [-1, 1], U = 3.4, u clamped to [-U, U] (erf(3.4) = 1 - 1.5e-6), and Q
// the degree-11 polynomial that interpolates erf(u) / u at the Chebyshev nodes in t (fitted for this file; the
// coefficients are those of the powers of t, all below 1 in size, so Horner's rule is stable in fp32).
// |error of Phi| < 1.6e-6 in fp32, three orders below bf16 resolution.
__device__ __forceinline__ unsigned long long norm_cdf2(unsigned long long z) {
  constexpr float U = 3.4f;
  const unsigned long long u = mul2(z, pk2(0.70710678118654752f, 0.70710678118654752f));
  const unsigned long long uc = pk2(fminf(fmaxf(lo2(u), -U), U), fminf(fmaxf(hi2(u), -U), U));
  const unsigned long long t = fma2(mul2(uc, uc), pk2(2.f / (U * U), 2.f / (U * U)), pk2(-1.f, -1.f));
  constexpr float c[12] = {4.156643398e-01f, -2.060884763e-01f, 1.495694051e-01f, -1.149434119e-01f, 8.608386700e-02f,
                           -6.136962761e-02f, 4.273188249e-02f, -2.607233935e-02f, 1.084438127e-02f, -5.875344802e-03f,
                           6.353731497e-03f, -2.781673617e-03f};
  unsigned long long acc = pk2(c[11], c[11]);
#pragma unroll
  for (int i = 10; i >= 0; --i) acc = fma2(acc, t, pk2(c[i], c[i]));
  return fma2(mul2(uc, acc), pk2(0.5f, 0.5f), pk2(0.5f, 0.5f));
}
// GeLU of a pair, in place.  VARIANT 0: z Phi(z); 1: the tanh form.
template <int VARIANT>
__device__ __forceinline__ void gelu_fwd2(float z0, float z1, float& h0, float& h1) {
  if (VARIANT == 0) {
    const unsigned long long z = pk2(z0, z1), h = mul2(z, norm_cdf2(z));
    h0 = lo2(h); h1 = hi2(h);
  } else {
    h0 = 0.5f * z0 * (1.f + tanhf(0.7978845608028654f * (z0 + 0.044715f * z0 * z0 * z0)));
    h1 = 0.5f * z1 * (1.f + tanhf(0.7978845608028654f * (z1 + 0.044715f * z1 * z1 * z1)));
  }
}
// GeLU'(z) of a pair.  VARIANT 0: Phi(z) + z phi(z), phi the normal density.
template <int VARIANT>
__device__ __forceinline__ void gelu_bwd2(float z0, float z1, float& g0, float& g1) {
  if (VARIANT == 0) {
    const unsigned long long z = pk2(z0, z1), Phi = norm_cdf2(z);
    // z exp(-z^2 / 2) / sqrt(2 pi)
    const unsigned long long zz = mul2(mul2(z, z), pk2(-0.72134752044448170f, -0.72134752044448170f));
    const unsigned long long e = pk2(exp2f(lo2(zz)), exp2f(hi2(zz)));
    const unsigned long long g = fma2(mul2(z, pk2(0.3989422804014327f, 0.3989422804014327f)), e, Phi);
    g0 = lo2(g); g1 = hi2(g);
  } else {
    const float a = 0.7978845608028654f;
    const float t0 = tanhf(a * (z0 + 0.044715f * z0 * z0 * z0)), t1 = tanhf(a * (z1 + 0.044715f * z1 * z1 * z1));
    g0 = 0.5f * (1.f + t0) + 0.5f * z0 * (1.f - t0 * t0) * a * (1.f + 3.f * 0.044715f * z0 * z0);
    g1 = 0.5f * (1.f + t1) + 0.5f * z1 * (1.f - t1 * t1) * a * (1.f + 3.f * 0.044715f * z1 * z1);
  }
}
__device__ __forceinline__ uint4 pack8(const float* f) {
  __nv_bfloat162 p0 = __floats2bfloat162_rn(f[0], f[1]), p1 = __floats2bfloat162_rn(f[2], f[3]);
  __nv_bfloat162 p2 = __floats2bfloat162_rn(f[4], f[5]), p3 = __floats2bfloat162_rn(f[6], f[7]);
  return make_uint4(*reinterpret_cast<unsigned*>(&p0), *reinterpret_cast<unsigned*>(&p1),
                    *reinterpret_cast<unsigned*>(&p2), *reinterpret_cast<unsigned*>(&p3));
}

// Ragged batches (token-choice routing leaves empty slots at the end of an expert's buffer): the k-blocks tile
// (b, mt) runs, 0 if it is skipped.  All three roles of a CTA call this with the same arguments and so agree.
__device__ __forceinline__ int tile_kblocks(const TcParams& p, int b, int mt, int tile_rows) {
  if (p.batch_rows == nullptr) return p.kblocks;
  const int rows = p.batch_rows[b];
  if (p.ragged == 1) return (mt > 0 && mt * tile_rows >= rows) ? 0 : p.kblocks;   // a batch's first row tile always runs
  const int kb = (rows + BK - 1) / BK;
  return kb < 1 ? 1 : (kb < p.kblocks ? kb : p.kblocks);
}

// ---------------------------------------------------------------------------------------------
// The kernel
// ---------------------------------------------------------------------------------------------
template <int BN, int EPI, int CTAS>
__global__ void __launch_bounds__(kThreads, 1)
gemm_tc_kernel(const __grid_constant__ CUtensorMap tmA, const __grid_constant__ CUtensorMap tmB,
               const __grid_constant__ CUtensorMap tmC, const __grid_constant__ CUtensorMap tmC2, const TcParams p) {
  constexpr int BNL = BN / CTAS;                    // rows of B this CTA loads
  constexpr int kMmaN = BN > 256 ? 256 : BN;        // columns of one MMA; a 512-wide tile takes two per K step
  constexpr int kBHalf = kMmaN / CTAS;              // rows of B this CTA contributes to one MMA
  constexpr bool kOneAcc = BN > 256;                // the tile fills tensor memory: one accumulator, no double buffering
  static_assert(BN <= 256 || CTAS == 2, "512-wide tiles are for CTA pairs");
  constexpr int TM = BM * CTAS;                     // rows of the tile the CTA (pair) works on
  constexpr bool kXchg = EPI == EPI_SOFTMAX && BN >= 128;            // the softmax epilogue's exchange area replaces a stage
  constexpr int kStaging = staging_bytes(BN, EPI);
  constexpr int S = num_stages(BNL, kStaging) - (kXchg ? 1 : 0);
  constexpr int kBBytes = BNL * BK * 2;
  constexpr int kStage = kABytes + kBBytes;
  constexpr int kCols = tmem_cols(BN, CTAS);
  extern __shared__ uint8_t smem_raw[];
  uint8_t* smem = (uint8_t*)(((uintptr_t)smem_raw + 1023) & ~(uintptr_t)1023);
  // barriers: full[S], empty[S], tmem_full[2], tmem_empty[2]; 256 bytes further on, with kXchg: [2][8 warps][32] float2, int[8]
  uint64_t* bars = (uint64_t*)(smem + S * kStage + kStaging);
  uint32_t* tmem_slot = (uint32_t*)(bars + 2 * S + 4);
  volatile int* abort_flag = (volatile int*)(tmem_slot + 1);
  const uint32_t full0 = smem_u32(bars), empty0 = full0 + 8 * S, tfull0 = empty0 + 8 * S, tempty0 = tfull0 + 16;
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const uint32_t rank = CTAS == 2 ? cluster_ctarank() : 0u;      // 0 = leader of the pair
  const int first_tile = blockIdx.x / CTAS, tile_step = gridDim.x / CTAS;

  if (threadIdx.x == 0) {
    // full: one arrival, the (leader's) producer announcing the bytes of the whole pair; tmem_empty: one per epilogue warp of the pair
    for (int s = 0; s < S; ++s) { mbar_init(full0 + 8 * s, 1); mbar_init(empty0 + 8 * s, 1); }
    for (int b = 0; b < 2; ++b) { mbar_init(tfull0 + 8 * b, 1); mbar_init(tempty0 + 8 * b, CTAS * kEpiWarps); }
    *abort_flag = 0;
    if constexpr (kXchg) {
      int* published = (int*)(smem + S * kStage + kStaging + 256 + 2 * kEpiWarps * 32 * 8);
      for (int w = 0; w < kEpiWarps; ++w) published[w] = 0;
    }
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  if (warp == 1) {
    asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(tmem_slot)), "r"(kCols) : "memory");
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
  }
  tc_fence_before();
  __syncthreads();
  if constexpr (CTAS == 2) cluster_sync_all();     // the peer's barriers exist before anything is sent to them
  tc_fence_after();
  const uint32_t tmem_base = *tmem_slot;
  const uint32_t smem_base = smem_u32(smem);
  bool gave_up = false;
  if (CTAS == 2 && tmem_base != 0) {               // cannot happen with all 512 columns taken; refuse rather than corrupt
    if (threadIdx.x == 0) { atomicExch(p.status + 1, 9); atomicExch(p.status, 5); }
    gave_up = true;
  }

  if (gave_up) {
    // nothing: fall through to the exit sequence
  } else if (warp == 0 && p.a_rows != nullptr) {
    // ------------------------------------------------------------------ TMA producer, A rows chosen through an index list
    // Eq. 3's X_in = P . X is not written: the stage's 128 x 64 block of A is filled by 32 row-indexed loads of four
    // rows each, one per lane (K-major A: the tile's 128 rows of M, the same for every k-block; MN-major A: two
    // 64-wide blocks of M times the k-block's 64 rows of K).  The shared-memory image is the one a box load of
    // X_in would have left (the 128-byte swizzle is a function of the shared-memory address).  Positions past the
    // end of the batch's list take its last entry: such rows of A meet either rows of C that are clipped (M) or
    // rows of B that the TMA unit zero-fills (K).  Lane 0 also loads B and announces the bytes, as the plain producer.
    int stage = 0; uint32_t phase = 0;
    const uint32_t leader_full0 = CTAS == 2 ? map_to_cta(full0, 0) : full0;
    const int nidx = p.a_mn ? p.K : p.M;               // stored rows of A per batch
    auto pick = [&](const int32_t* list, int pos) {
      const int r = __ldg(list + min(pos, nidx - 1));
      return idx_ok(r, 0, p.a_rows_total, p.status) ? r : 0;
    };
    for (int tile = first_tile; tile < p.total_tiles && !gave_up; tile += tile_step) {
      const int b = tile / (p.tiles_m * p.tiles_n);
      const int mt = p.n_fast ? (tile / p.tiles_n) % p.tiles_m : tile % p.tiles_m;
      const int nt = p.n_fast ? tile % p.tiles_n : (tile / p.tiles_m) % p.tiles_n;
      const int m0 = mt * TM + (int)rank * BM, n0 = nt * BN + (int)rank * kBHalf;
      const int32_t* rows_b = p.a_rows + (int64_t)b * p.a_rows_batch;
      int ri[4];
      const int rbase = p.a_mn ? 4 * (lane & 15) : m0 + 4 * lane;
#pragma unroll
      for (int j = 0; j < 4; ++j) ri[j] = pick(rows_b, rbase + j);
      for (int kb = 0; kb < p.kblocks; ++kb) {
        const bool ok = mbar_wait(empty0 + 8 * stage, phase ^ 1, abort_flag, p.status, 1);
        if (!__all_sync(0xffffffffu, ok)) { gave_up = true; break; }
        const uint32_t sa = smem_base + stage * kStage, sb = sa + kABytes;
        const int k0 = kb * BK;
        const uint32_t bar = (CTAS == 2 ? leader_full0 : full0) + 8 * stage;
        if (lane == 0) {
          if constexpr (CTAS == 2) {
            if (rank == 0) mbar_expect_tx(full0 + 8 * stage, 2 * kStage);
            if (p.b_mn) {
#pragma unroll
              for (int j = 0; j < BNL / 64; ++j)
                tma_load_3d_pair(sb + j * (BK * 128), &tmB, bar, n0 + (64 * j / kBHalf) * kMmaN + 64 * j % kBHalf, k0, b);
            } else {
#pragma unroll
              for (int j = 0; j < BNL / kBHalf; ++j) tma_load_3d_pair(sb + j * (kBHalf * 128), &tmB, bar, k0, n0 + j * kMmaN, b);
            }
          } else {
            mbar_expect_tx(bar, kStage);
            if (p.b_mn) {
#pragma unroll
              for (int j = 0; j < BNL / 64; ++j) tma_load_3d(sb + j * (BK * 128), &tmB, bar, n0 + 64 * j, k0, b);
            } else {
              tma_load_3d(sb, &tmB, bar, k0, n0, b);
            }
          }
        }
        __syncwarp();                                    // the announcement is made before any of the warp's copies can land
        const uint32_t dst = p.a_mn ? sa + (lane >> 4) * (BK * 128) + (lane & 15) * 512 : sa + lane * 512;
        const int col = p.a_mn ? m0 + 64 * (lane >> 4) : k0;
        if constexpr (CTAS == 2) tma_gather4_pair(dst, &tmA, bar, col, ri[0], ri[1], ri[2], ri[3]);
        else tma_gather4(dst, &tmA, bar, col, ri[0], ri[1], ri[2], ri[3]);
        if (p.a_mn && kb + 1 < p.kblocks) {              // the next k-block's rows of K, fetched while this one lands
#pragma unroll
          for (int j = 0; j < 4; ++j) ri[j] = pick(rows_b, (kb + 1) * BK + rbase + j);
        }
        if (++stage == S) { stage = 0; phase ^= 1; }
      }
    }
  } else if (warp == 0) {
    // ------------------------------------------------------------------ TMA producer
    if (lane == 0) {
      int stage = 0; uint32_t phase = 0;
      const uint32_t leader_full0 = CTAS == 2 ? map_to_cta(full0, 0) : full0;
      for (int tile = first_tile; tile < p.total_tiles && !gave_up; tile += tile_step) {
        const int b = tile / (p.tiles_m * p.tiles_n);
        const int mt = p.n_fast ? (tile / p.tiles_n) % p.tiles_m : tile % p.tiles_m;
        const int nt = p.n_fast ? tile % p.tiles_n : (tile / p.tiles_m) % p.tiles_n;
        // B columns of this CTA: per 256-wide MMA the pair's two halves of kBHalf columns each, side by side
        const int m0 = mt * TM + (int)rank * BM, n0 = nt * BN + (int)rank * kBHalf;
        const int kblocks = tile_kblocks(p, b, mt, TM);
        for (int kb = 0; kb < kblocks; ++kb) {
          if (!mbar_wait(empty0 + 8 * stage, phase ^ 1, abort_flag, p.status, 1)) { gave_up = true; break; }
          const uint32_t sa = smem_base + stage * kStage, sb = sa + kABytes;
          const int k0 = kb * BK + (p.k_split ? b * p.K : 0);
          const int bc = p.k_split ? 0 : b;          // third coordinate of the operand maps
          if constexpr (CTAS == 2) {
            // The leader's barrier collects both halves: its producer announces the pair's bytes, the
            // peer's copies simply complete on it (they may land before the announcement; the phase
            // cannot end before the leader's arrival and a byte count of zero).
            const uint32_t bar = leader_full0 + 8 * stage;
            if (rank == 0) mbar_expect_tx(full0 + 8 * stage, 2 * kStage);
            if (p.a_mn) {
#pragma unroll
              for (int j = 0; j < BM / 64; ++j) tma_load_3d_pair(sa + j * (BK * 128), &tmA, bar, m0 + 64 * j, k0, bc);
            } else {
              tma_load_3d_pair(sa, &tmA, bar, k0, m0, bc);
            }
            if (p.b_mn) {
#pragma unroll
              for (int j = 0; j < BNL / 64; ++j)
                tma_load_3d_pair(sb + j * (BK * 128), &tmB, bar, n0 + (64 * j / kBHalf) * kMmaN + 64 * j % kBHalf, k0, bc);
            } else {
#pragma unroll
              for (int j = 0; j < BNL / kBHalf; ++j) tma_load_3d_pair(sb + j * (kBHalf * 128), &tmB, bar, k0, n0 + j * kMmaN, bc);
            }
          } else {
            const uint32_t bar = full0 + 8 * stage;
            mbar_expect_tx(bar, kStage);
            if (p.a_mn) {                       // stored [K][M]: boxes of 64 (M) x 64 (K)
#pragma unroll
              for (int j = 0; j < BM / 64; ++j) tma_load_3d(sa + j * (BK * 128), &tmA, bar, m0 + 64 * j, k0, bc);
            } else {                            // stored [M][K]: one box 64 (K) x 128 (M)
              tma_load_3d(sa, &tmA, bar, k0, m0, bc);
            }
            if (p.b_mn) {
#pragma unroll
              for (int j = 0; j < BNL / 64; ++j) tma_load_3d(sb + j * (BK * 128), &tmB, bar, n0 + 64 * j, k0, bc);
            } else {
              tma_load_3d(sb, &tmB, bar, k0, n0, bc);
            }
          }
          if (++stage == S) { stage = 0; phase ^= 1; }
        }
      }
    }
  } else if (warp == 1) {
    // ------------------------------------------------------------------ MMA issuer (the leader's, in a pair)
    if (lane == 0 && rank == 0) {
      const uint32_t idesc = (1u << 4) | (1u << 7) | (1u << 10) | ((uint32_t)p.a_mn << 15) | ((uint32_t)p.b_mn << 16) |
                             ((uint32_t)(kMmaN >> 3) << 17) | ((uint32_t)(TM >> 4) << 24);
      // K-major: 8-row groups 1024 B apart, 32 B per K step inside the swizzle atom.
      // MN-major: 64-wide blocks BK*128 B apart (LBO), 8-row K groups 1024 B apart (SBO), 2 groups per K step.
      const uint32_t a_lbo = p.a_mn ? BK * 128 : 16, b_lbo = p.b_mn ? BK * 128 : 16;
      const uint32_t a_step = p.a_mn ? 2048 : 32, b_step = p.b_mn ? 2048 : 32;
      int stage = 0; uint32_t phase = 0; int it = 0;
      for (int tile = first_tile; tile < p.total_tiles && !gave_up; tile += tile_step) {
        const int kblocks = tile_kblocks(p, tile / (p.tiles_m * p.tiles_n),
                                         p.n_fast ? (tile / p.tiles_n) % p.tiles_m : tile % p.tiles_m, TM);
        if (kblocks == 0) continue;                  // a tile of empty slots: no accumulator is used
        const int buf = kOneAcc ? 0 : it & 1; const uint32_t use = (uint32_t)(kOneAcc ? it : it >> 1);
        ++it;
        if (!mbar_wait(tempty0 + 8 * buf, (use & 1) ^ 1, abort_flag, p.status, 2)) { gave_up = true; break; }
        tc_fence_after();
        const uint32_t d_tmem = tmem_base + buf * BN;
        for (int kb = 0; kb < kblocks; ++kb) {
          if (!mbar_wait(full0 + 8 * stage, phase, abort_flag, p.status, 3)) { gave_up = true; break; }
          tc_fence_after();
          const uint32_t sa = smem_base + stage * kStage, sb = sa + kABytes;
#pragma unroll
          for (int kk = 0; kk < BK / UK; ++kk) {
            const uint64_t ad = make_desc(sa + kk * a_step, a_lbo, 1024);
            const uint64_t bd = make_desc(sb + kk * b_step, b_lbo, 1024);
            if constexpr (CTAS == 2) tc_mma_pair(d_tmem, ad, bd, idesc, (kb | kk) != 0);
            else tc_mma(d_tmem, ad, bd, idesc, (kb | kk) != 0);
            if constexpr (kOneAcc) {                 // the tile's second 256 columns: same A, the next kBHalf rows of B
              const uint64_t bd2 = make_desc(sb + kBHalf * 128 + kk * b_step, b_lbo, 1024);
              tc_mma_pair(d_tmem + kMmaN, ad, bd2, idesc, (kb | kk) != 0);
            }
          }
          // the stage is free (in both CTAs) once these MMAs have read it
          if constexpr (CTAS == 2) tc_commit_pair(empty0 + 8 * stage); else tc_commit(empty0 + 8 * stage);
          if (++stage == S) { stage = 0; phase ^= 1; }
        }
        if (!gave_up) {                              // accumulator complete
          if constexpr (CTAS == 2) tc_commit_pair(tfull0 + 8 * buf); else tc_commit(tfull0 + 8 * buf);
        }
      }
    }
  } else {
    // ------------------------------------------------------------------ epilogue, one tile row per thread
    const int q = warp & 3;                        // TMEM lane quarter this warp may read
    const int half = (warp - 2) >> 2;              // which half of the tile's columns this warp handles
    int it = 0;
    uint32_t nchunk = 0;                           // chunks this warp has stored so far: picks the staging buffer
    const uint32_t tempty_leader = CTAS == 2 ? map_to_cta(tempty0, 0) : tempty0;
    for (int tile = first_tile; tile < p.total_tiles; tile += tile_step) {
      const int b = tile / (p.tiles_m * p.tiles_n);
      const int mt = p.n_fast ? (tile / p.tiles_n) % p.tiles_m : tile % p.tiles_m;
      const int nt = p.n_fast ? tile % p.tiles_n : (tile / p.tiles_m) % p.tiles_n;
      if (tile_kblocks(p, b, mt, TM) == 0) continue; // a tile of empty slots: nothing was accumulated, nothing is stored
      const int buf = kOneAcc ? 0 : it & 1; const uint32_t use = (uint32_t)(kOneAcc ? it : it >> 1);
      const bool ok = mbar_wait(tfull0 + 8 * buf, use & 1, abort_flag, p.status, 4);
      if constexpr (EPI == EPI_STORE) {
        // the four warps of a column half meet at named barriers below: they leave together or not at all (every one
        // of them gets here, its wait being bounded)
        if (!half_all(half, ok)) { gave_up = true; break; }
      } else {
        if (!__all_sync(0xffffffffu, ok)) { gave_up = true; break; }
      }
      tc_fence_after();
      const int row = mt * TM + (int)rank * BM + q * 32 + lane;
      const bool row_ok = row < p.M;
      const uint32_t taddr = tmem_base + ((uint32_t)(q * 32) << 16) + buf * BN;
      const int n0 = nt * BN;
      const int64_t obase = (int64_t)b * p.batch_c + (int64_t)row * p.ldc;
      if constexpr (EPI == EPI_SOFTMAX) {
        // Eq. 2: softmax over the N = E columns of each row; columns >= N are padding.  A thread owns one
        // row.  With BN >= 128 the two warps of a lane quarter take half of the columns each and exchange
        // their (max, sum) through shared memory.  First sweep over tensor memory: running max and sum
        // of exp(x - max); second sweep: exp(x - max) / sum, staged and stored like any fp32 result.
        constexpr bool kSplit = BN >= 128;
        constexpr int kColsPerWarp = kSplit ? BN / 2 : BN;
        const int cbeg = kSplit ? half * kColsPerWarp : 0;
        const bool active = kSplit || half == 0;
        uint8_t* stg = smem + S * kStage + (warp - 2) * kStagingPerWarp;
        const uint32_t stg_s = smem_u32(stg);
        const int r0 = mt * TM + (int)rank * BM + q * 32;
        float mx = -INFINITY, sum = 0.f;
        if (active) {
#pragma unroll 1
          for (int c0 = cbeg; c0 < cbeg + kColsPerWarp && c0 < p.N; c0 += 32) {
            uint32_t r[32]; tc_ld32(taddr + c0, r);
            float cm = -INFINITY;
#pragma unroll
            for (int j = 0; j < 32; ++j) if (c0 + j < p.N) cm = fmaxf(cm, __uint_as_float(r[j]));
            const float mn = fmaxf(mx, cm);
            float part = 0.f;
#pragma unroll
            for (int j = 0; j < 32; ++j) if (c0 + j < p.N) part += __expf(__uint_as_float(r[j]) - mn);
            sum = sum * __expf(mx - mn) + part;
            mx = mn;
          }
        }
        if constexpr (kSplit) {
          // The partner's (max, sum) comes through a slot in shared memory, one per warp and tile parity, with
          // a per-warp counter of published tiles.  A slot is rewritten two tiles later, which the partner's
          // release of the accumulator (it precedes that tile's MMAs) orders after its read.  The wait is bounded.
          float2* xch = reinterpret_cast<float2*>(smem + S * kStage + kStaging + 256);
          volatile int* published = reinterpret_cast<volatile int*>(xch + 2 * kEpiWarps * 32);
          const int me = warp - 2, partner = me ^ 4;
          xch[((it & 1) * kEpiWarps + me) * 32 + lane] = make_float2(mx, sum);
          __threadfence_block();
          __syncwarp();
          if (lane == 0) published[me] = it + 1;
          bool seen = published[partner] >= it + 1;
          if (!seen) {
            const unsigned long long t0 = globaltimer();
            for (uint32_t spin = 1; !seen; ++spin) {
              seen = published[partner] >= it + 1;
              if (!seen && (spin & 63u) == 0 && (*abort_flag || globaltimer() - t0 > kWaitNs)) break;
            }
          }
          if (!__all_sync(0xffffffffu, seen)) {
            if (lane == 0) { *abort_flag = 1; atomicExch(p.status + 1, 7); atomicExch(p.status, 5); }
            gave_up = true; break;
          }
          __threadfence_block();
          const float2 o = xch[((it & 1) * kEpiWarps + partner) * 32 + lane];
          const float mn = fmaxf(mx, o.x);
          sum = sum * __expf(mx - mn) + (o.y > 0.f ? o.y * __expf(o.x - mn) : 0.f);
          mx = mn;
        }
        const float inv = 1.f / sum;
        const int sw = lane & 7;
        if (active) {
#pragma unroll 1
          for (int c0 = cbeg; c0 < cbeg + kColsPerWarp && c0 < p.N; c0 += 32, ++nchunk) {
            uint32_t r[32]; tc_ld32(taddr + c0, r);
            uint8_t* bufp = stg + (nchunk & 1) * 4096;
            if (lane == 0) bulk_wait_read<1>();
            __syncwarp();
#pragma unroll
            for (int j = 0; j < 8; ++j) {
              float4 o;
              o.x = __expf(__uint_as_float(r[4 * j]) - mx) * inv; o.y = __expf(__uint_as_float(r[4 * j + 1]) - mx) * inv;
              o.z = __expf(__uint_as_float(r[4 * j + 2]) - mx) * inv; o.w = __expf(__uint_as_float(r[4 * j + 3]) - mx) * inv;
              *reinterpret_cast<float4*>(bufp + lane * 128 + ((j ^ sw) << 4)) = o;
            }
            fence_async_smem();
            __syncwarp();
            if (lane == 0 && r0 < p.M) { tma_store_3d(&tmC, stg_s + (nchunk & 1) * 4096, c0, r0, 0); bulk_commit(); }
          }
        }
      } else {
        // Results leave through shared memory and the TMA unit.  A warp owns 32 rows and kColsPerWarp columns
        // of the tile and works on chunks whose rows are 128 bytes long (64 bf16 or 32 fp32 columns): each
        // thread converts its row of the chunk and writes it with the 128-byte swizzle (conflict-free) into one
        // of the warp's two 4 KiB staging buffers, one lane issues a bulk tensor store, which writes whole
        // 128-byte lines and clips what overhangs M or N.  The buffers alternate from chunk to chunk (across
        // tiles too); one is reused once the store issued two chunks earlier has read it.
        uint8_t* stg = smem + S * kStage + (warp - 2) * kStagingPerWarp;
        const uint32_t stg_s = smem_u32(stg);
        const int r0 = mt * TM + (int)rank * BM + q * 32;
        const int sw = lane & 7;
        constexpr int kColsPerWarp = BN >= 128 ? BN / 2 : BN;      // a 64-wide tile is drained by the first four warps alone
        const bool active = half * kColsPerWarp < BN;
        if constexpr (EPI == EPI_STORE_F32) {
#pragma unroll 1
          for (int c0 = half * kColsPerWarp; active && c0 < (half + 1) * kColsPerWarp; c0 += 32, ++nchunk) {
            if (n0 + c0 >= p.N) break;             // uniform across the warp
            uint32_t r[32]; tc_ld32(taddr + c0, r);
            if (p.bias != nullptr) {               // the bias term of Eq. 3's second product: the same 32 values for every row
              const bf16* bp = p.bias + (int64_t)b * p.N + n0 + c0;
#pragma unroll
              for (int j = 0; j < 4; ++j) {
                if (n0 + c0 + 8 * j < p.N) {
                  const uint4 bv = __ldg(reinterpret_cast<const uint4*>(bp + 8 * j));
                  const unsigned w[4] = {bv.x, bv.y, bv.z, bv.w};
#pragma unroll
                  for (int e = 0; e < 4; ++e) {
                    r[8 * j + 2 * e] = __float_as_uint(__uint_as_float(r[8 * j + 2 * e]) + __uint_as_float(w[e] << 16));
                    r[8 * j + 2 * e + 1] = __float_as_uint(__uint_as_float(r[8 * j + 2 * e + 1]) + __uint_as_float(w[e] & 0xFFFF0000u));
                  }
                }
              }
            }
            uint8_t* bufp = stg + (nchunk & 1) * 4096;
            if (lane == 0) bulk_wait_read<1>();
            __syncwarp();
#pragma unroll
            for (int j = 0; j < 8; ++j)
              *reinterpret_cast<uint4*>(bufp + lane * 128 + ((j ^ sw) << 4)) =
                  make_uint4(r[4 * j], r[4 * j + 1], r[4 * j + 2], r[4 * j + 3]);
            fence_async_smem();
            __syncwarp();
            if (lane == 0 && r0 < p.M) { tma_store_3d(&tmC, stg_s + (nchunk & 1) * 4096, n0 + c0, r0, b); bulk_commit(); }
          }
        } else {
#pragma unroll 1
          for (int c0 = half * kColsPerWarp; active && c0 < (half + 1) * kColsPerWarp; c0 += 64, ++nchunk) {
            if (n0 + c0 >= p.N) break;             // uniform across the warp
            uint32_t r[64];
            tc_ld32_issue(taddr + c0, r); tc_ld32_issue(taddr + c0 + 32, r + 32); tc_ld_wait();
            if constexpr (EPI == EPI_GELU) {
              if (p.bias != nullptr) {             // Z = X_in . W1 + b1: the same 64 values for every row
                const bf16* bp = p.bias + (int64_t)b * p.N + n0 + c0;
#pragma unroll
                for (int j = 0; j < 8; ++j) {
                  if (n0 + c0 + 8 * j < p.N) {
                    const uint4 bv = __ldg(reinterpret_cast<const uint4*>(bp + 8 * j));
                    const unsigned w[4] = {bv.x, bv.y, bv.z, bv.w};
#pragma unroll
                    for (int e = 0; e < 4; ++e) {
                      r[8 * j + 2 * e] = __float_as_uint(__uint_as_float(r[8 * j + 2 * e]) + __uint_as_float(w[e] << 16));
                      r[8 * j + 2 * e + 1] = __float_as_uint(__uint_as_float(r[8 * j + 2 * e + 1]) + __uint_as_float(w[e] & 0xFFFF0000u));
                    }
                  }
                }
              }
              // both buffers are written: Z into the first, H = GeLU(Z) into the second
              if (lane == 0) bulk_wait_read<0>();
              __syncwarp();
              // one uniform branch on the GeLU form around the whole chunk: inside it only that form is evaluated
              auto convert = [&](auto variant) {
#pragma unroll
                for (int j = 0; j < 8; ++j) {
                  float z[8], h[8];
#pragma unroll
                  for (int e = 0; e < 8; e += 2) {
                    z[e] = __uint_as_float(r[8 * j + e]); z[e + 1] = __uint_as_float(r[8 * j + e + 1]);
                    gelu_fwd2<decltype(variant)::value>(z[e], z[e + 1], h[e], h[e + 1]);
                  }
                  if (!p.skip_c) *reinterpret_cast<uint4*>(stg + lane * 128 + ((j ^ sw) << 4)) = pack8(z);
                  *reinterpret_cast<uint4*>(stg + 4096 + lane * 128 + ((j ^ sw) << 4)) = pack8(h);
                }
              };
              if (p.gelu == 0) convert(std::integral_constant<int, 0>{}); else convert(std::integral_constant<int, 1>{});
              fence_async_smem();
              __syncwarp();
              if (lane == 0 && r0 < p.M) {
                if (!p.skip_c) tma_store_3d(&tmC, stg_s, n0 + c0, r0, b);
                tma_store_3d(&tmC2, stg_s + 4096, n0 + c0, r0, b);
                bulk_commit();
              }
            } else {
              if constexpr (EPI == EPI_GELU_GRAD) {
                // dZ = acc * GeLU'(Z): this thread's 64 values of Z (128 bytes of its row)
                const bf16* zp = p.Zin + obase + n0 + c0;
                uint4 zv[8];
#pragma unroll
                for (int j = 0; j < 8; ++j) {
                  zv[j] = make_uint4(0, 0, 0, 0);
                  if (row_ok && n0 + c0 + 8 * j < p.N) zv[j] = *reinterpret_cast<const uint4*>(zp + 8 * j);
                }
                auto scale = [&](auto variant) {             // one uniform branch on the GeLU form, as above
#pragma unroll
                  for (int j = 0; j < 8; ++j) {
                    const unsigned zw[4] = {zv[j].x, zv[j].y, zv[j].z, zv[j].w};
#pragma unroll
                    for (int e = 0; e < 4; ++e) {
                      float g0, g1;
                      gelu_bwd2<decltype(variant)::value>(__uint_as_float(zw[e] << 16), __uint_as_float(zw[e] & 0xFFFF0000u), g0, g1);
                      r[8 * j + 2 * e] = __float_as_uint(__uint_as_float(r[8 * j + 2 * e]) * g0);
                      r[8 * j + 2 * e + 1] = __float_as_uint(__uint_as_float(r[8 * j + 2 * e + 1]) * g1);
                    }
                  }
                };
                if (p.gelu == 0) scale(std::integral_constant<int, 0>{}); else scale(std::integral_constant<int, 1>{});
              }
              if constexpr (EPI == EPI_ADD_SLOTS) {
                // this thread's row gains the rows of its slots (128 bytes of each), in slot order
                if (row_ok) {
                  int qa = p.row_ptr[row], qb = p.row_ptr[row + 1];
                  if (!idx_ok(qa, 0, p.slots_total + 1, p.status) || !idx_ok(qb, qa, p.slots_total + 1, p.status)) qa = qb = 0;
                  for (int qq = qa; qq < qb; ++qq) {
                    const int sid = p.slots[qq];
                    if (!idx_ok(sid, 0, p.slots_total, p.status)) continue;
                    const bf16* src = p.rows + (int64_t)sid * p.ld_rows + n0 + c0;
#pragma unroll
                    for (int j = 0; j < 8; ++j) {
                      if (n0 + c0 + 8 * j < p.N) {
                        const uint4 v = *reinterpret_cast<const uint4*>(src + 8 * j);
                        const unsigned w[4] = {v.x, v.y, v.z, v.w};
#pragma unroll
                        for (int e = 0; e < 4; ++e) {
                          r[8 * j + 2 * e] = __float_as_uint(__uint_as_float(r[8 * j + 2 * e]) + __uint_as_float(w[e] << 16));
                          r[8 * j + 2 * e + 1] = __float_as_uint(__uint_as_float(r[8 * j + 2 * e + 1]) + __uint_as_float(w[e] & 0xFFFF0000u));
                        }
                      }
                    }
                  }
                }
              }
              if constexpr (EPI == EPI_STORE) {
                // Plain results leave in boxes of 128 rows: the four warps of this column half fill one 16 KiB buffer
                // (two per half, alternating), one thread stores it.  Four stores per 128 x 256 block instead of sixteen:
                // the weight gradients, which write a tile's 64 KiB per eight k-blocks, gain 3 % (8 % alone in a loop).
                uint8_t* hb = smem + S * kStage + half * (4 * kStagingPerWarp) + (nchunk & 1) * 16384;
                const bool leader = q == 0 && lane == 0;
                if (leader) bulk_wait_read<1>();     // the store that last read this buffer (two chunks ago) is through with it
                half_sync(half);
#pragma unroll
                for (int j = 0; j < 8; ++j) {
                  float f[8];
#pragma unroll
                  for (int e = 0; e < 8; ++e) f[e] = __uint_as_float(r[8 * j + e]);
                  *reinterpret_cast<uint4*>(hb + (q * 32 + lane) * 128 + ((j ^ sw) << 4)) = pack8(f);
                }
                fence_async_smem();
                half_sync(half);
                const int rt0 = mt * TM + (int)rank * BM;
                if (leader && rt0 < p.M) { tma_store_3d(&tmC, smem_u32(hb), n0 + c0, rt0, b); bulk_commit(); }
              } else {
                uint8_t* bufp = stg + (nchunk & 1) * 4096;
                if (lane == 0) bulk_wait_read<1>();  // the other buffer's store may still be in flight
                __syncwarp();
#pragma unroll
                for (int j = 0; j < 8; ++j) {
                  float f[8];
#pragma unroll
                  for (int e = 0; e < 8; ++e) f[e] = __uint_as_float(r[8 * j + e]);
                  *reinterpret_cast<uint4*>(bufp + lane * 128 + ((j ^ sw) << 4)) = pack8(f);
                }
                fence_async_smem();
                __syncwarp();
                if (lane == 0 && r0 < p.M) { tma_store_3d(&tmC, stg_s + (nchunk & 1) * 4096, n0 + c0, r0, b); bulk_commit(); }
              }
            }
          }
        }
      }
      tc_fence_before();
      __syncwarp();                                // every lane's tcgen05.ld has completed
      if (lane == 0) {                             // one arrival per warp frees the accumulator
        if constexpr (CTAS == 2) mbar_arrive_cluster(tempty_leader + 8 * buf); else mbar_arrive(tempty0 + 8 * buf);
      }
      ++it;                                        // tiles this CTA has worked on (skipped ones do not count)
    }
  }

  // ------------------------------------------------------------------ orderly exit
  if (warp >= 2 && lane == 0) bulk_wait_all();     // this warp's stores have left shared memory and are complete
  if (*abort_flag) {                               // let copies and MMAs still in flight drain
    const unsigned long long t0 = globaltimer();
    while (globaltimer() - t0 < 200000ull) __nanosleep(1000);
  }
  __syncwarp();
  tc_fence_before();
  __syncthreads();
  if constexpr (CTAS == 2) cluster_sync_all();     // the peer no longer reads this CTA's shared or writes its tensor memory
  if (warp == 1) {
    tc_fence_after();
    asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem_base), "r"(kCols) : "memory");
  }
}

// ---------------------------------------------------------------------------------------------
// Host side
// ---------------------------------------------------------------------------------------------
PFN_cuTensorMapEncodeTiled_v12000 get_encode() {
  static PFN_cuTensorMapEncodeTiled_v12000 fn = nullptr;
  static std::once_flag once;
  std::call_once(once, [] {
    void* p = nullptr; cudaDriverEntryPointQueryResult qr;
    if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &p, cudaEnableDefault, &qr) == cudaSuccess &&
        qr == cudaDriverEntryPointSuccess)
      fn = (PFN_cuTensorMapEncodeTiled_v12000)p;
  });
  return fn;
}

// Tensor map over a matrix stored [batches][rows][inner] with row pitch ld and batch pitch bs (elements).
bool make_map(CUtensorMap* tm, const void* base, int64_t inner, int64_t rows, int64_t batches, int64_t ld, int64_t bs,
              int box_inner, int box_rows, bool f32 = false, CUtensorMapSwizzle swz = CU_TENSOR_MAP_SWIZZLE_128B) {
  auto enc = get_encode();
  if (!enc) return false;
  const cuuint64_t es_bytes = f32 ? 4 : 2;
  cuuint64_t dims[3] = {(cuuint64_t)inner, (cuuint64_t)rows, (cuuint64_t)batches};
  cuuint64_t strides[2] = {(cuuint64_t)ld * es_bytes, (cuuint64_t)(batches > 1 ? bs : rows * ld) * es_bytes};
  cuuint32_t box[3] = {(cuuint32_t)box_inner, (cuuint32_t)box_rows, 1};
  cuuint32_t es[3] = {1, 1, 1};
  return enc(tm, f32 ? CU_TENSOR_MAP_DATA_TYPE_FLOAT32 : CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 3, const_cast<void*>(base),
             dims, strides, box, es, CU_TENSOR_MAP_INTERLEAVE_NONE, swz, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
             CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

// Tensor map for row-indexed loads (tile::gather4) from a matrix [rows][inner] with row pitch ld: two dimensions,
// a box of 64 elements of one row.
bool make_gather_map(CUtensorMap* tm, const void* base, int64_t inner, int64_t rows, int64_t ld) {
  auto enc = get_encode();
  if (!enc) return false;
  cuuint64_t dims[2] = {(cuuint64_t)inner, (cuuint64_t)rows};
  cuuint64_t strides[1] = {(cuuint64_t)ld * 2};
  cuuint32_t box[2] = {64, 1};
  cuuint32_t es[2] = {1, 1};
  return enc(tm, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, const_cast<void*>(base), dims, strides, box, es,
             CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
             CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

// 512 columns per tile for a CTA pair on a long contraction with a plain store; else 256 columns when the
// tile is a CTA pair's; a single CTA (M <= 128: few rows per expert, the product
// streams the weights) does better with 128, whose smaller stages leave room for five of them instead of three
int pick_bn(const TcGemmArgs& g, int pairs) {
  // Eq. 2's softmax runs over all N = E columns of a row inside one tile's epilogue: the tile must hold them all
  if (g.epi == EPI_SOFTMAX) return g.N > 128 ? 256 : (g.N > 64 ? 128 : 64);
  if (g.M > BM && g.N >= 512 && g.K >= kWideMinK && g.epi == EPI_STORE) {
    // waves of tiles over the CTA pairs, a 512-column tile counted as 1.92 of a 256-column one (its saving in
    // fill less its epilogue in the open): padding of N to 512 and a thinner last wave can cost more than that
    const int64_t rows = (int64_t)((g.M + 2 * BM - 1) / (2 * BM)) * g.batches;
    const int64_t narrow = (rows * ((g.N + 255) / 256) + pairs - 1) / pairs, wide = (rows * ((g.N + 511) / 512) + pairs - 1) / pairs;
    if (wide * 192 <= narrow * 100) return 512;
  }
  return (g.N > 128 && g.M > BM) ? 256 : (g.N > 64 ? 128 : 64);
}
// Two CTAs per tile when a tile of 256 rows is not mostly padding and the pair's B halves are whole 64-wide blocks.
int pick_ctas(const TcGemmArgs& g, int bn) { return (bn >= 128 && g.M > BM) ? 2 : 1; }

template <int BN, int EPI, int CTAS>
cudaError_t launch_one(const CUtensorMap& ta, const CUtensorMap& tb, const CUtensorMap& tc, const CUtensorMap& tc2,
                       const TcParams& p, cudaStream_t st) {
  // the split softmax trades one operand stage for its exchange area (4 KiB + counters), see the kernel
  constexpr int smem = num_stages(BN / CTAS, staging_bytes(BN, EPI)) * stage_bytes(BN / CTAS) + staging_bytes(BN, EPI) + 1024 + 256;
  auto kern = gemm_tc_kernel<BN, EPI, CTAS>;
  cudaError_t e = cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, smem);
  if (e != cudaSuccess) return e;
  int dev = 0, sms = 148;
  cudaGetDevice(&dev);
  cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev);
  cudaLaunchConfig_t cfg; memset(&cfg, 0, sizeof(cfg));
  cfg.blockDim = dim3(kThreads); cfg.dynamicSmemBytes = smem; cfg.stream = st;
  cudaLaunchAttribute attr[1];
  int groups = sms / CTAS;                           // CTAs (or pairs) that run at once
  if (CTAS == 2) {
    attr[0].id = cudaLaunchAttributeClusterDimension;
    attr[0].val.clusterDim.x = 2; attr[0].val.clusterDim.y = 1; attr[0].val.clusterDim.z = 1;
    cfg.attrs = attr; cfg.numAttrs = 1;
    // pairs the device can hold at once, per device; host threads may race to fill an entry, with the same value
    static std::atomic<int> max_pairs[64];
    if (dev >= 0 && dev < 64) {
      int mp = max_pairs[dev].load(std::memory_order_relaxed);
      if (mp == 0) {
        cfg.gridDim = dim3(2 * groups);
        int nc = 0;
        mp = (cudaOccupancyMaxActiveClusters(&nc, kern, &cfg) == cudaSuccess && nc > 0) ? nc : groups;
        max_pairs[dev].store(mp, std::memory_order_relaxed);
      }
      if (mp < groups) groups = mp;
    }
  }
  if (p.total_tiles < groups) groups = p.total_tiles;
  cfg.gridDim = dim3(groups * CTAS);
  count_launch();
  return cudaLaunchKernelEx(&cfg, kern, ta, tb, tc, tc2, p);
}

template <int EPI>
cudaError_t launch_bn(int bn, int ctas, const CUtensorMap& ta, const CUtensorMap& tb, const CUtensorMap& tc, const CUtensorMap& tc2,
                      const TcParams& p, cudaStream_t st) {
  {
    if (ctas == 2) {
      if constexpr (EPI == EPI_STORE || EPI == EPI_STORE_F32) {
        if (bn == 512) return launch_one<512, EPI, 2>(ta, tb, tc, tc2, p, st);
      }
      if (bn == 256) return launch_one<256, EPI, 2>(ta, tb, tc, tc2, p, st);
      return launch_one<128, EPI, 2>(ta, tb, tc, tc2, p, st);
    }
  }
  if (bn == 256) return launch_one<256, EPI, 1>(ta, tb, tc, tc2, p, st);
  if (bn == 128) return launch_one<128, EPI, 1>(ta, tb, tc, tc2, p, st);
  return launch_one<64, EPI, 1>(ta, tb, tc, tc2, p, st);
}

}  // namespace

bool tc_gemm_supported(const TcGemmArgs& g) {
  if (g.M < 1 || g.N < 1 || g.K < 1 || g.batches < 1) return false;
  if (g.lda % 8 || g.ldb % 8 || g.ldc % 8 || g.N % 8) return false;            // 16-byte rows and vector stores
  if (g.batches > 1 && (g.batch_a % 8 || g.batch_b % 8 || g.batch_c % 8)) return false;
  if (((uintptr_t)g.A | (uintptr_t)g.B) & 15) return false;
  if (g.epi == EPI_SOFTMAX && (g.N > 256 || g.batches != 1)) return false;
  if (g.k_split && (g.K % BK || g.k_total < 1 || !g.c_f32 || g.epi != EPI_STORE)) return false;
  if (g.epi == EPI_ADD_SLOTS && (g.batches != 1 || g.c_f32 || !g.row_ptr || !g.slots || !g.rows || g.ld_rows % 8 ||
                                 ((uintptr_t)g.rows & 15))) return false;
  if ((int64_t)g.lda * 2 >= ((int64_t)1 << 40) || (int64_t)g.ldb * 2 >= ((int64_t)1 << 40)) return false;
  if (g.batch_rows && (g.k_split || (g.ragged != 1 && g.ragged != 2))) return false;
  if (g.bias && (((uintptr_t)g.bias & 15) || g.k_split || !(g.epi == EPI_GELU || (g.epi == EPI_STORE && g.c_f32)))) return false;
  if (g.a_rows && (g.k_split || g.batch_rows || g.epi == EPI_SOFTMAX || g.a_rows_total < 1 || g.a_rows_total >= ((int64_t)1 << 31))) return false;
  return true;
}

cudaError_t launch_gemm_tc(const TcGemmArgs& g, cudaStream_t st) {
  int dev = 0, sms = 148;
  cudaGetDevice(&dev);
  cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev);
  const int bn = pick_bn(g, sms / 2);
  const int ctas = pick_ctas(g, bn);
  const int bnl = bn / ctas;                         // rows of B one CTA loads
  CUtensorMap ta, tb;
  // A: K-major [M rows][K inner], box 64 x 128;  MN-major [K rows][M inner], box 64 x 64
  // operand maps: with k_split both are single matrices whose K extent is the whole contraction
  const int64_t kext = g.k_split ? g.k_total : g.K;
  const int64_t ob = g.k_split ? 1 : g.batches;
  const bool oka = g.a_rows ? make_gather_map(&ta, g.A, g.a_mn_major ? g.M : g.K, g.a_rows_total, g.lda)
                 : g.a_mn_major ? make_map(&ta, g.A, g.M, kext, ob, g.lda, g.batch_a, 64, BK)
                                : make_map(&ta, g.A, kext, g.M, ob, g.lda, g.batch_a, BK, BM);
  const bool okb = g.b_mn_major ? make_map(&tb, g.B, g.N, kext, ob, g.ldb, g.batch_b, 64, BK)
                                : make_map(&tb, g.B, kext, g.N, ob, g.ldb, g.batch_b, BK, bnl > 128 ? 128 : bnl);
  if (!oka || !okb) return cudaErrorInvalidValue;
  // outputs leave through TMA stores of chunks of 32 rows x 128 bytes (64 bf16 or 32 fp32 columns)
  CUtensorMap tc = ta, tc2 = ta;
  if (g.epi == EPI_SOFTMAX) {
    if (!make_map(&tc, g.S, g.N, g.M, 1, g.ldc, 0, 32, 32, true)) return cudaErrorInvalidValue;
  } else {
    const void* cbase = (g.epi == EPI_GELU && !g.C) ? g.C2 : g.C;     // without C its map is never used: any valid one will do
    // plain bf16 results are stored in boxes of 128 rows (a column half's four warps together), the rest in boxes of 32
    if (!make_map(&tc, cbase, g.N, g.M, g.batches, g.ldc, g.batch_c, g.c_f32 ? 32 : 64, (g.epi == EPI_STORE && !g.c_f32) ? 128 : 32,
                  g.c_f32 != 0)) return cudaErrorInvalidValue;
    if (g.epi == EPI_GELU && !make_map(&tc2, g.C2, g.N, g.M, g.batches, g.ldc, g.batch_c, 64, 32)) return cudaErrorInvalidValue;
  }
  TcParams p;
  p.M = g.M; p.N = g.N; p.K = g.K; p.batches = g.batches; p.a_mn = g.a_mn_major; p.b_mn = g.b_mn_major;
  p.tiles_m = (g.M + BM * ctas - 1) / (BM * ctas); p.tiles_n = (g.N + bn - 1) / bn;
  p.total_tiles = p.tiles_m * p.tiles_n * g.batches; p.kblocks = (g.K + BK - 1) / BK;
  p.gelu = g.gelu;
  p.Zin = (const bf16*)g.Zin;
  p.ldc = g.ldc; p.batch_c = g.batch_c; p.status = g.status;
  p.k_split = g.k_split; p.skip_c = (g.epi == EPI_GELU && !g.C) ? 1 : 0;
  // Tile order.  Tiles running at the same time are consecutive ones.  Along M (default) they share the B tile,
  // which for the expert FFNs is the weight matrix: it is then read from HBM once.  When the output is larger
  // than the operands (short K: the weight gradients) the tiles run along N instead, so that what is written at
  // one time is whole rows of C rather than 512-byte pieces 2*N bytes apart, and they share the A tile.
  p.n_fast = (int64_t)g.M * g.N > ((int64_t)g.M + g.N) * g.K ? 1 : 0;
  p.row_ptr = g.row_ptr; p.slots = g.slots; p.rows = (const bf16*)g.rows; p.ld_rows = g.ld_rows; p.slots_total = g.slots_total;
  p.batch_rows = g.batch_rows; p.ragged = g.ragged;
  p.bias = (const bf16*)g.bias;
  p.a_rows = g.a_rows; p.a_rows_batch = g.a_rows_batch; p.a_rows_total = (int)g.a_rows_total;
  switch (g.epi) {
    case EPI_STORE: return g.c_f32 ? launch_bn<EPI_STORE_F32>(bn, ctas, ta, tb, tc, tc2, p, st)
                                   : launch_bn<EPI_STORE>(bn, ctas, ta, tb, tc, tc2, p, st);
    case EPI_GELU: return launch_bn<EPI_GELU>(bn, ctas, ta, tb, tc, tc2, p, st);
    case EPI_GELU_GRAD: return launch_bn<EPI_GELU_GRAD>(bn, ctas, ta, tb, tc, tc2, p, st);
    case EPI_ADD_SLOTS: return launch_bn<EPI_ADD_SLOTS>(bn, ctas, ta, tb, tc, tc2, p, st);
    case EPI_SOFTMAX: return launch_bn<EPI_SOFTMAX>(bn, ctas, ta, tb, tc, tc2, p, st);
  }
  return cudaErrorInvalidValue;
}

}  // namespace ecmoe
