// Expert choice with at most b experts per token (Section 3.3): the matrix A [e, n] of
//
//     max <S^T, A> + lambda H(A)   s.t.  rows sum to k,  columns sum to at most b,  0 <= A <= 1
//
// by Dykstra's algorithm with Kullback-Leibler projections onto the three sets in turn, a fixed number of
// rounds.  The projections are rescalings and a clip, so the iteration runs on L = log A, stored token-major
// ([n, e], like S) beside the log correction factors of the column set (one per token) and of the box set
// (one per entry):
//
//     rows:     L[t, i] += log k - logsumexp_t L[:, i]
//     columns:  B = L[t, :] + qc[t];  m = min(0, log b - logsumexp_i B);  L[t, :] = B + m;  qc[t] = -m
//     box:      B = L + qb;  L = min(B, 0);  qb = B - L
//
// A warp owns a token (its e values, a few per lane), so the column and box steps need only warp shuffles; the
// row step needs a sum over all tokens, which a round prepares for the next: every CTA leaves (max, sum of exp)
// of its tokens per expert, and the CTAs each combine those in a fixed order (so the result does not depend on
// scheduling) before they touch their tokens.  Two forms:
//   - resident: one cooperative launch for all rounds; a warp keeps log A and the factors of its (at most 8 /
//     experts-per-lane) tokens in registers, the CTAs meet at a grid barrier once per round and only the row
//     partials go through memory.  Used whenever the tokens fit (up to about 19 k tokens at 64 experts);
//   - resident in shared memory: the same launch with the state in the CTA's shared memory, for up to about
//     2.4 M entries per device (16384 tokens x 128 experts, 65536 x 32);
//   - one launch per round with the state (2 x 4 bytes per entry) in global memory, where it stays in L2 at
//     the layer sizes.  For everything else.
// Either way a round costs latency (a barrier or a launch, one round trip for the partials, the reduction
// trees), not bandwidth.  Routing groups are independent problems (grid.y).
#include "internal.h"

#include <cooperative_groups.h>
#include <math.h>

namespace ecmoe {

namespace {

namespace cg = cooperative_groups;

constexpr int kCapThreads = 1024;
constexpr int kCapWarps = kCapThreads / 32;
constexpr int kCapMaxE = 256;
constexpr int kCapLoads = 4;                         // partials a thread of the row step has in flight 
constexpr int kCapBatch = 4;                         // tokens of a warp whose loads are in flight together (fewer with many experts per lane)
constexpr int kCapResident = 8;                      // (tokens per warp) x (experts per lane) the resident form holds:
                                                     // log A and the box factors of that many entries in a lane's registers

// (m, s) stands for s * exp(m); the sum of two such numbers (the same bits whichever operand comes first)
__device__ __forceinline__ void lse_add(float& m, float& s, float m2, float s2) {
  if (s2 == 0.f) return;
  if (s == 0.f) { m = m2; s = s2; return; }
  if (m2 > m) { s = s * __expf(m - m2) + s2; m = m2; } else { s += s2 * __expf(m2 - m); }
}
// butterfly over `width` adjacent lanes (a power of two): every lane ends with the same sum
__device__ __forceinline__ void lse_butterfly(float& m, float& s, int width) {
  for (int o = width >> 1; o > 0; o >>= 1) {
    const float m2 = __shfl_xor_sync(0xffffffffu, m, o), s2 = __shfl_xor_sync(0xffffffffu, s, o);
    lse_add(m, s, m2, s2);
  }
}

// Shared memory of a CTA: wpart [warps][E] float2 | shift [E] float
__device__ __forceinline__ float* shift_of(float2* smem, int E) { return reinterpret_cast<float*>(smem + kCapWarps * E); }

// shift[i] = log k - log(sum over the group's tokens of exp L[:, i]) from the partials the CTAs of group g left.
// P adjacent lanes share an expert: each combines every P-th CTA's partial in ascending order (loads several at
// a time, kCapLoads in flight), a butterfly joins them.  Every thread of the CTA calls this.
// The partials were written by other CTAs, in the resident forms by the same launch: they are read from L2
// (ld.global.cg), never through a read-only or L1 path that could hold the values of two rounds ago.
__device__ __forceinline__ void row_shifts(const float2* part_in, int g, int bpg, int E, float log_k, float* shift) {
  int P = 32;
  while (P * E > kCapThreads) P >>= 1;               // E <= 256: P >= 4
  const int i = threadIdx.x / P, p0 = threadIdx.x % P;
  float m = 0.f, s = 0.f;
  if (i < E) {
    for (int q = p0; q < bpg; q += kCapLoads * P) {
      float2 v[kCapLoads];
#pragma unroll
      for (int u = 0; u < kCapLoads; ++u) {
        const int qq = q + u * P;
        v[u] = qq < bpg ? __ldcg(part_in + ((int64_t)g * E + i) * bpg + qq) : make_float2(0.f, 0.f);   // adjacent lanes, adjacent CTAs
      }
#pragma unroll
      for (int u = 0; u < kCapLoads; ++u) lse_add(m, s, v[u].x, v[u].y);
    }
  }
  lse_butterfly(m, s, P);                            // whole warps take part: P divides 32
  if (i < E && p0 == 0) shift[i] = log_k - (m + __logf(s));
  __syncthreads();
}

// The CTA's (max, sum of exp) per expert from the lanes' running values; warp w joins experts w, w + 32, ...
template <int EPL>
__device__ __forceinline__ void publish_partials(const float (&pm)[EPL], const float (&ps)[EPL], float2* wpart, int E,
                                                 float2* __restrict__ part_out, int g, int bpg, int blk) {
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  __syncthreads();                                   // the previous use of wpart and shift is over
#pragma unroll
  for (int j = 0; j < EPL; ++j) if (lane + 32 * j < E) wpart[warp * E + lane + 32 * j] = make_float2(pm[j], ps[j]);
  __syncthreads();
  for (int i = warp; i < E; i += kCapWarps) {
    float2 v = wpart[lane * E + i];
    lse_butterfly(v.x, v.y, 32);
    if (lane == 0) part_out[((int64_t)g * E + i) * bpg + blk] = v;     // expert-major: the row step reads along the CTAs
  }
}

// One token, one round after the row step: columns, then the box.  x: log A of the token's experts held by this
// lane (already shifted by the row step), qb / qc: log correction factors.  Returns nothing; updates in place.
template <int EPL>
__device__ __forceinline__ void token_round(float (&x)[EPL], float (&qb)[EPL], float& qc, int lane, int E, float log_b) {
  // After the row step every entry is at most k (its row sums to k), so exp cannot overflow and the column sum
  // needs no shift by the maximum; a column so small that the sum underflows is far below b and stays as it is.
  float sum = 0.f;
#pragma unroll
  for (int j = 0; j < EPL; ++j) if (lane + 32 * j < E) sum += __expf(x[j]);
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) sum += __shfl_xor_sync(0xffffffffu, sum, o);
  const float m = fminf(0.f, log_b - (__logf(sum) + qc));             // a column above b is scaled down to b
#pragma unroll
  for (int j = 0; j < EPL; ++j) {
    if (lane + 32 * j < E) {
      const float B = x[j] + qc + m + qb[j];
      const float v = fminf(B, 0.f);                                 // entries above 1 are clipped
      qb[j] = B - v;
      x[j] = v;
    }
  }
  qc = -m;
}

// ---- one launch per round ------------------------------------------------------------------------
// phase 0: L = S / lambda and its row partials.  phase 1: one round (rows, columns, box) and the row
// partials of its result; `first` treats the correction factors as 1 without reading them, `last`
// also writes A = exp(L).
template <int EPL>
__global__ void __launch_bounds__(kCapThreads)
capped_round_kernel(const float* __restrict__ S, float* __restrict__ L, float* __restrict__ qb, float* __restrict__ qc,
                    float* __restrict__ A, const float2* __restrict__ part_in, float2* __restrict__ part_out,
                    int64_t ng, int E, float inv_lambda, float log_k, float log_b, int phase, int first, int last) {
  constexpr int kBatch = EPL >= 8 ? 1 : (EPL >= 4 ? 2 : kCapBatch);   // so that a batch fits the 64 registers of a thread
  extern __shared__ float2 cap_smem[];
  float* shift = shift_of(cap_smem, E);
  const int g = blockIdx.y, bpg = gridDim.x, blk = blockIdx.x;
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  float pm[EPL], ps[EPL];
#pragma unroll
  for (int j = 0; j < EPL; ++j) { pm[j] = 0.f; ps[j] = 0.f; }
  // A warp takes its tokens kBatch at a time: the loads of a batch are issued together (they do not depend on
  // the row sums, so the first batch's are in flight while the CTA combines the partials), the arithmetic
  // follows token by token in ascending order.
  const int64_t stride = (int64_t)bpg * kCapWarps;
  float x[kBatch][EPL], qbv[kBatch][EPL], qcv[kBatch];
  auto load_batch = [&](int64_t tb) {
#pragma unroll
    for (int u = 0; u < kBatch; ++u) {
      const int64_t t = tb + u * stride;
      const int64_t tok = (int64_t)g * ng + t, row = tok * E;
      qcv[u] = 0.f;
#pragma unroll
      for (int j = 0; j < EPL; ++j) {
        const int i = lane + 32 * j;
        const bool ok = t < ng && i < E;
        x[u][j] = !ok ? -INFINITY : (phase == 0 ? S[row + i] * inv_lambda : L[row + i]);
        qbv[u][j] = (ok && phase == 1 && !first) ? qb[row + i] : 0.f;
      }
      if (t < ng && phase == 1 && !first) qcv[u] = qc[tok];
    }
  };
  int64_t tb = (int64_t)blk * kCapWarps + warp;
  load_batch(tb);                                    // loads nothing for a warp without tokens
  if (phase == 1) row_shifts(part_in, g, bpg, E, log_k, shift);       // every thread of the CTA gets here
  while (tb < ng) {
#pragma unroll
    for (int u = 0; u < kBatch; ++u) {
      const int64_t t = tb + u * stride;
      if (t < ng) {                                                    // uniform across the warp
        const int64_t tok = (int64_t)g * ng + t, row = tok * E;
        if (phase == 1) {
#pragma unroll
          for (int j = 0; j < EPL; ++j) if (lane + 32 * j < E) x[u][j] += shift[lane + 32 * j];     // rows sum to k
          token_round<EPL>(x[u], qbv[u], qcv[u], lane, E, log_b);
          if (lane == 0) qc[tok] = qcv[u];
        }
#pragma unroll
        for (int j = 0; j < EPL; ++j) {
          const int i = lane + 32 * j;
          if (i < E) {
            L[row + i] = x[u][j];
            if (phase == 1) qb[row + i] = qbv[u][j];
            if (last) A[row + i] = __expf(x[u][j]);
            if (phase == 0) lse_add(pm[j], ps[j], x[u][j], 1.f);
            else ps[j] += __expf(x[u][j]);           // after a round: entries at most 1, row sums well above underflow
          }
        }
      }
    }
    tb += kBatch * stride;
    if (tb < ng) load_batch(tb);
  }
  publish_partials<EPL>(pm, ps, cap_smem, E, part_out, g, bpg, blk);
}

// ---- resident: all rounds in one cooperative launch ------------------------------------------------
// Needs ng <= TPW * gridDim.x * warps per CTA; every CTA calls the grid barrier iters times.
template <int EPL, int TPW>
__global__ void __launch_bounds__(kCapThreads)
capped_resident_kernel(const float* __restrict__ S, float* __restrict__ A, float2* __restrict__ part0, float2* __restrict__ part1,
                       int64_t ng, int E, float inv_lambda, float log_k, float log_b, int iters) {
  extern __shared__ float2 cap_smem[];
  float* shift = shift_of(cap_smem, E);
  cg::grid_group grid = cg::this_grid();
  const int g = blockIdx.y, bpg = gridDim.x, blk = blockIdx.x;
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int64_t stride = (int64_t)bpg * kCapWarps, t0 = (int64_t)blk * kCapWarps + warp;
  float x[TPW][EPL], qb[TPW][EPL], qc[TPW], pm[EPL], ps[EPL];
#pragma unroll
  for (int j = 0; j < EPL; ++j) { pm[j] = 0.f; ps[j] = 0.f; }
#pragma unroll
  for (int u = 0; u < TPW; ++u) {
    const int64_t t = t0 + u * stride, row = ((int64_t)g * ng + t) * E;
    qc[u] = 0.f;
#pragma unroll
    for (int j = 0; j < EPL; ++j) {
      const int i = lane + 32 * j;
      qb[u][j] = 0.f;
      x[u][j] = (t < ng && i < E) ? S[row + i] * inv_lambda : -INFINITY;
      if (t < ng && i < E) lse_add(pm[j], ps[j], x[u][j], 1.f);
    }
  }
  publish_partials<EPL>(pm, ps, cap_smem, E, part0, g, bpg, blk);
  for (int it = 0; it < iters; ++it) {
    grid.sync();                                     // every CTA's partials of the previous pass are in memory
    row_shifts((it & 1) ? part1 : part0, g, bpg, E, log_k, shift);
#pragma unroll
    for (int j = 0; j < EPL; ++j) { pm[j] = 0.f; ps[j] = 0.f; }
#pragma unroll
    for (int u = 0; u < TPW; ++u) {
      if (t0 + u * stride < ng) {                    // uniform across the warp
#pragma unroll
        for (int j = 0; j < EPL; ++j) if (lane + 32 * j < E) x[u][j] += shift[lane + 32 * j];       // rows sum to k
        token_round<EPL>(x[u], qb[u], qc[u], lane, E, log_b);
#pragma unroll
        for (int j = 0; j < EPL; ++j) if (lane + 32 * j < E) ps[j] += __expf(x[u][j]);      // entries at most 1
      }
    }
    if (it + 1 < iters) publish_partials<EPL>(pm, ps, cap_smem, E, (it & 1) ? part0 : part1, g, bpg, blk);
  }
#pragma unroll
  for (int u = 0; u < TPW; ++u) {
    const int64_t t = t0 + u * stride, row = ((int64_t)g * ng + t) * E;
#pragma unroll
    for (int j = 0; j < EPL; ++j) if (t < ng && lane + 32 * j < E) A[row + lane + 32 * j] = __expf(x[u][j]);
  }
}

// The same with the state in shared memory instead of registers, for groups whose tokens do not fit the registers:
// behind wpart and shift come log A and the box factors of the warp's tokens ([warp][token][2][E]) and the column
// factors ([warp][token]).  A warp touches only its own part, so no barrier guards it.
template <int EPL>
__global__ void __launch_bounds__(kCapThreads)
capped_resident_smem_kernel(const float* __restrict__ S, float* __restrict__ A, float2* __restrict__ part0,
                            float2* __restrict__ part1, int64_t ng, int E, float inv_lambda, float log_k, float log_b,
                            int iters, int tpw) {
  extern __shared__ float2 cap_smem[];
  float* shift = shift_of(cap_smem, E);
  cg::grid_group grid = cg::this_grid();
  const int g = blockIdx.y, bpg = gridDim.x, blk = blockIdx.x;
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int64_t stride = (int64_t)bpg * kCapWarps, t0 = (int64_t)blk * kCapWarps + warp;
  float* mine = shift + E + (size_t)warp * tpw * 2 * E;            // this warp's tokens: [token][log A | box factor][E]
  float* my_qc = shift + E + (size_t)kCapWarps * tpw * 2 * E + warp * tpw;
  float pm[EPL], ps[EPL];
#pragma unroll
  for (int j = 0; j < EPL; ++j) { pm[j] = 0.f; ps[j] = 0.f; }
  for (int u = 0; u < tpw; ++u) {
    const int64_t t = t0 + u * stride, row = ((int64_t)g * ng + t) * E;
    if (t < ng) {                                    // uniform across the warp
#pragma unroll
      for (int j = 0; j < EPL; ++j) {
        const int i = lane + 32 * j;
        if (i < E) {
          const float v = S[row + i] * inv_lambda;
          mine[(2 * u) * E + i] = v; mine[(2 * u + 1) * E + i] = 0.f;
          lse_add(pm[j], ps[j], v, 1.f);
        }
      }
      if (lane == 0) my_qc[u] = 0.f;
    }
  }
  publish_partials<EPL>(pm, ps, cap_smem, E, part0, g, bpg, blk);
  for (int it = 0; it < iters; ++it) {
    grid.sync();                                     // every CTA's partials of the previous pass are in memory
    row_shifts((it & 1) ? part1 : part0, g, bpg, E, log_k, shift);
#pragma unroll
    for (int j = 0; j < EPL; ++j) { pm[j] = 0.f; ps[j] = 0.f; }
    for (int u = 0; u < tpw; ++u) {
      if (t0 + u * stride < ng) {                    // uniform across the warp
        float x[EPL], qb[EPL];
#pragma unroll
        for (int j = 0; j < EPL; ++j) {
          const int i = lane + 32 * j;
          x[j] = i < E ? mine[(2 * u) * E + i] + shift[i] : -INFINITY;                               // rows sum to k
          qb[j] = i < E ? mine[(2 * u + 1) * E + i] : 0.f;
        }
        float qc = my_qc[u];
        __syncwarp();                                // every lane has read the column factor before lane 0 rewrites it
        token_round<EPL>(x, qb, qc, lane, E, log_b);
        if (lane == 0) my_qc[u] = qc;
#pragma unroll
        for (int j = 0; j < EPL; ++j) {
          const int i = lane + 32 * j;
          if (i < E) { mine[(2 * u) * E + i] = x[j]; mine[(2 * u + 1) * E + i] = qb[j]; ps[j] += __expf(x[j]); }
        }
      }
    }
    if (it + 1 < iters) publish_partials<EPL>(pm, ps, cap_smem, E, (it & 1) ? part0 : part1, g, bpg, blk);
  }
  for (int u = 0; u < tpw; ++u) {
    const int64_t t = t0 + u * stride, row = ((int64_t)g * ng + t) * E;
#pragma unroll
    for (int j = 0; j < EPL; ++j) if (t < ng && lane + 32 * j < E) A[row + lane + 32 * j] = __expf(mine[(2 * u) * E + lane + 32 * j]);
  }
}

__global__ void gather_gate_kernel(const float* __restrict__ S, const int32_t* __restrict__ I, float* __restrict__ G,
                                   int64_t slots_total, int64_t k, int E, int64_t n, int* status) {
  for (int64_t s = (int64_t)blockIdx.x * blockDim.x + threadIdx.x; s < slots_total; s += (int64_t)gridDim.x * blockDim.x) {
    const int t = I[s];
    G[s] = idx_ok(t, 0, n, status) ? S[(int64_t)t * E + (int)(s / k)] : 0.f;
  }
}

int blocks_per_group(int64_t ng, int groups, int sms) {
  int64_t b = sms / groups;
  const int64_t most = (ng + kCapWarps - 1) / kCapWarps;            // at least one token per warp
  if (b > most) b = most;
  return (int)(b < 1 ? 1 : b);
}
// The partials are sized for the largest grid any device could ask for, so the layout does not depend on the device.
constexpr int kCapMaxBlocks = 1024;

size_t align256(size_t b) { return (b + 255) & ~(size_t)255; }
size_t cap_smem_bytes(int E) { return (size_t)kCapWarps * E * 8 + (size_t)E * 4; }      // at most 65 KiB

struct ResidentArgs {
  const float* S; float* A; float2* part0; float2* part1; int64_t ng; int E; float inv_lambda, log_k, log_b; int iters;
};
template <int EPL, int TPW>
cudaError_t launch_resident(ResidentArgs a, dim3 grid, int sms, bool* fits, cudaStream_t st) {
  auto kern = capped_resident_kernel<EPL, TPW>;
  const size_t smem = cap_smem_bytes(a.E);
  if (smem > 48 * 1024 && cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, 66 * 1024) != cudaSuccess)
    return cudaErrorInvalidValue;
  int per_sm = 0;
  if (cudaOccupancyMaxActiveBlocksPerMultiprocessor(&per_sm, kern, kCapThreads, smem) != cudaSuccess) return cudaErrorInvalidValue;
  *fits = (int64_t)per_sm * sms >= (int64_t)grid.x * grid.y;         // a grid barrier needs every CTA on the device at once
  if (!*fits) return cudaSuccess;
  void* args[] = {&a.S, &a.A, &a.part0, &a.part1, &a.ng, &a.E, &a.inv_lambda, &a.log_k, &a.log_b, &a.iters};
  count_launch();
  return cudaLaunchCooperativeKernel((void*)kern, grid, dim3(kCapThreads), args, smem, st);
}
template <int EPL>
cudaError_t launch_resident_tpw(int tpw, ResidentArgs a, dim3 grid, int sms, bool* fits, cudaStream_t st) {
  if constexpr (EPL <= 8) if (tpw <= 1) return launch_resident<EPL, 1>(a, grid, sms, fits, st);
  if constexpr (EPL <= 4) if (tpw <= 2) return launch_resident<EPL, 2>(a, grid, sms, fits, st);
  if constexpr (EPL <= 2) if (tpw <= 4) return launch_resident<EPL, 4>(a, grid, sms, fits, st);
  if constexpr (EPL <= 1) if (tpw <= 8) return launch_resident<EPL, 8>(a, grid, sms, fits, st);
  *fits = false;
  return cudaSuccess;
}

constexpr size_t kCapSmemLimit = 200 * 1024;         // of a CTA's 227 KiB
template <int EPL>
cudaError_t launch_resident_smem(ResidentArgs a, int tpw, dim3 grid, int sms, bool* fits, cudaStream_t st) {
  auto kern = capped_resident_smem_kernel<EPL>;
  const size_t smem = cap_smem_bytes(a.E) + (size_t)kCapWarps * tpw * (2 * a.E + 1) * 4;
  *fits = false;
  if (smem > kCapSmemLimit) return cudaSuccess;
  if (cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)kCapSmemLimit) != cudaSuccess) return cudaErrorInvalidValue;
  int per_sm = 0;
  if (cudaOccupancyMaxActiveBlocksPerMultiprocessor(&per_sm, kern, kCapThreads, smem) != cudaSuccess) return cudaErrorInvalidValue;
  *fits = (int64_t)per_sm * sms >= (int64_t)grid.x * grid.y;
  if (!*fits) return cudaSuccess;
  void* args[] = {&a.S, &a.A, &a.part0, &a.part1, &a.ng, &a.E, &a.inv_lambda, &a.log_k, &a.log_b, &a.iters, &tpw};
  count_launch();
  return cudaLaunchCooperativeKernel((void*)kern, grid, dim3(kCapThreads), args, smem, st);
}

}  // namespace

// scratch: L [n, E] | qb [n, E] | qc [n] | two sets of row partials
size_t capped_scratch_bytes(int64_t n, int E, int groups) {
  const size_t blocks = (size_t)(groups > kCapMaxBlocks ? groups : kCapMaxBlocks);
  return 2 * align256((size_t)n * E * 4) + align256((size_t)n * 4) + 2 * align256(blocks * E * sizeof(float2));
}

cudaError_t launch_capped_assignment(const float* S, int64_t ng, int E, int64_t kg, int groups, int b, int iters,
                                     float lambda, float* A, void* scratch, cudaStream_t st) {
  if (E > kCapMaxE || iters < 1 || b < 1 || !(lambda > 0.f)) return cudaErrorInvalidValue;
  const int64_t n = ng * groups;
  char* p = (char*)scratch;
  float* L = (float*)p; p += align256((size_t)n * E * 4);
  float* qb = (float*)p; p += align256((size_t)n * E * 4);
  float* qc = (float*)p; p += align256((size_t)n * 4);
  const size_t blocks = (size_t)(groups > kCapMaxBlocks ? groups : kCapMaxBlocks);
  float2* part[2] = {(float2*)p, (float2*)(p + align256(blocks * E * sizeof(float2)))};
  int dev = 0, sms = 148, coop = 0;
  cudaGetDevice(&dev);
  cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev);
  cudaDeviceGetAttribute(&coop, cudaDevAttrCooperativeLaunch, dev);
  int bpg = blocks_per_group(ng, groups, sms);
  if ((int64_t)bpg * groups > (int64_t)blocks) bpg = (int)(blocks / groups);
  const dim3 grid(bpg, groups);
  const float inv_lambda = 1.f / lambda, log_k = logf((float)kg), log_b = logf((float)b);
  const int epl = E <= 32 ? 1 : (E <= 64 ? 2 : (E <= 128 ? 4 : 8));
  const int64_t tpw = (ng + (int64_t)bpg * kCapWarps - 1) / ((int64_t)bpg * kCapWarps);
  if (coop && tpw * epl <= kCapResident) {
    ResidentArgs a{S, A, part[0], part[1], ng, E, inv_lambda, log_k, log_b, iters};
    bool fits = false;
    cudaError_t e = epl == 1 ? launch_resident_tpw<1>((int)tpw, a, grid, sms, &fits, st)
                  : epl == 2 ? launch_resident_tpw<2>((int)tpw, a, grid, sms, &fits, st)
                  : epl == 4 ? launch_resident_tpw<4>((int)tpw, a, grid, sms, &fits, st)
                             : launch_resident_tpw<8>((int)tpw, a, grid, sms, &fits, st);
    if (e != cudaSuccess) return e;
    if (fits) return cudaGetLastError();
  }
  if (coop && tpw * epl > kCapResident && tpw <= 1024) {             // too many entries for registers: try shared memory
    ResidentArgs a{S, A, part[0], part[1], ng, E, inv_lambda, log_k, log_b, iters};
    bool fits = false;
    cudaError_t e = epl == 1 ? launch_resident_smem<1>(a, (int)tpw, grid, sms, &fits, st)
                  : epl == 2 ? launch_resident_smem<2>(a, (int)tpw, grid, sms, &fits, st)
                  : epl == 4 ? launch_resident_smem<4>(a, (int)tpw, grid, sms, &fits, st)
                             : launch_resident_smem<8>(a, (int)tpw, grid, sms, &fits, st);
    if (e != cudaSuccess) return e;
    if (fits) return cudaGetLastError();
  }
  const size_t smem = cap_smem_bytes(E);
  if (smem > 48 * 1024 &&                            // E > 180: more than the default limit
      cudaFuncSetAttribute(capped_round_kernel<8>, cudaFuncAttributeMaxDynamicSharedMemorySize, 66 * 1024) != cudaSuccess)
    return cudaErrorInvalidValue;
  auto round = [&](int phase, int first, int last, const float2* in, float2* out) {
    count_launch();
    if (E <= 32) capped_round_kernel<1><<<grid, kCapThreads, smem, st>>>(S, L, qb, qc, A, in, out, ng, E, inv_lambda, log_k, log_b, phase, first, last);
    else if (E <= 64) capped_round_kernel<2><<<grid, kCapThreads, smem, st>>>(S, L, qb, qc, A, in, out, ng, E, inv_lambda, log_k, log_b, phase, first, last);
    else if (E <= 128) capped_round_kernel<4><<<grid, kCapThreads, smem, st>>>(S, L, qb, qc, A, in, out, ng, E, inv_lambda, log_k, log_b, phase, first, last);
    else capped_round_kernel<8><<<grid, kCapThreads, smem, st>>>(S, L, qb, qc, A, in, out, ng, E, inv_lambda, log_k, log_b, phase, first, last);
  };
  round(0, 0, 0, nullptr, part[0]);
  for (int it = 0; it < iters; ++it) round(1, it == 0, it == iters - 1, part[it & 1], part[(it + 1) & 1]);
  return cudaGetLastError();
}

cudaError_t launch_gather_gate(const float* S, const int32_t* I, float* G, int64_t slots_total, int64_t k, int E,
                               int64_t n, int* status, cudaStream_t st) {
  count_launch();
  const int64_t blocks = (slots_total + 255) / 256;
  gather_gate_kernel<<<(unsigned)(blocks > 1184 ? 1184 : blocks), 256, 0, st>>>(S, I, G, slots_total, k, E, n, status);
  return cudaGetLastError();
}

}  // namespace ecmoe
