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
// One launch per round.  A warp owns a token (its e values, a few per lane), so the column and box steps need
// only warp shuffles; the row step needs a sum over all tokens, which a round prepares for the next: every
// CTA leaves (max, sum of exp) of its tokens per expert, and the next launch's CTAs each combine those in CTA
// order (fixed, so the result does not depend on scheduling) before they touch their tokens.  The state is
// 2 x 4 bytes per (token, expert) and stays in L2 at the layer sizes; the chain is bound by launch and
// reduction latency (about 10 us per round), not by bandwidth.  Routing groups are independent problems
// (grid.y).
#include "internal.h"

#include <math.h>

namespace ecmoe {

namespace {

constexpr int kCapThreads = 512;
constexpr int kCapWarps = kCapThreads / 32;
constexpr int kCapMaxE = 256;

// (m, s) stands for s * exp(m); the sum of two such numbers
__device__ __forceinline__ void lse_add(float& m, float& s, float m2, float s2) {
  if (s2 == 0.f) return;
  if (s == 0.f) { m = m2; s = s2; return; }
  if (m2 > m) { s = s * expf(m - m2) + s2; m = m2; } else { s += s2 * expf(m2 - m); }
}

// phase 0: L = S / lambda and its row partials.  phase 1: one round (rows, columns, box) and the row
// partials of its result; `first` treats the correction factors as 1 without reading them, `last`
// also writes A = exp(L).
template <int EPL>
__global__ void __launch_bounds__(kCapThreads)
capped_round_kernel(const float* __restrict__ S, float* __restrict__ L, float* __restrict__ qb, float* __restrict__ qc,
                    float* __restrict__ A, const float2* __restrict__ part_in, float2* __restrict__ part_out,
                    int64_t ng, int E, float inv_lambda, float log_k, float log_b, int phase, int first, int last) {
  __shared__ float shift[kCapMaxE];
  __shared__ float2 wpart[kCapWarps][kCapMaxE];
  const int g = blockIdx.y, bpg = gridDim.x, blk = blockIdx.x;
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  if (phase == 1) {
    for (int i = threadIdx.x; i < E; i += kCapThreads) {
      float m = 0.f, s = 0.f;
      for (int q = 0; q < bpg; ++q) {
        const float2 p = part_in[((int64_t)g * bpg + q) * E + i];
        lse_add(m, s, p.x, p.y);
      }
      shift[i] = log_k - (m + logf(s));
    }
    __syncthreads();
  }
  float pm[EPL], ps[EPL];
#pragma unroll
  for (int j = 0; j < EPL; ++j) { pm[j] = 0.f; ps[j] = 0.f; }
  for (int64_t t = (int64_t)blk * kCapWarps + warp; t < ng; t += (int64_t)bpg * kCapWarps) {
    const int64_t tok = (int64_t)g * ng + t, row = tok * E;
    float x[EPL];
    if (phase == 0) {
#pragma unroll
      for (int j = 0; j < EPL; ++j) {
        const int i = lane + 32 * j;
        x[j] = i < E ? S[row + i] * inv_lambda : -INFINITY;
        if (i < E) L[row + i] = x[j];
      }
    } else {
      float mx = -INFINITY;
#pragma unroll
      for (int j = 0; j < EPL; ++j) {
        const int i = lane + 32 * j;
        x[j] = i < E ? L[row + i] + shift[i] : -INFINITY;          // rows sum to k
        mx = fmaxf(mx, x[j]);
      }
#pragma unroll
      for (int o = 16; o > 0; o >>= 1) mx = fmaxf(mx, __shfl_xor_sync(0xffffffffu, mx, o));
      float sum = 0.f;
#pragma unroll
      for (int j = 0; j < EPL; ++j) if (lane + 32 * j < E) sum += expf(x[j] - mx);
#pragma unroll
      for (int o = 16; o > 0; o >>= 1) sum += __shfl_xor_sync(0xffffffffu, sum, o);
      const float q = first ? 0.f : qc[tok];
      const float m = fminf(0.f, log_b - (mx + logf(sum) + q));    // a column above b is scaled down to b
      if (lane == 0) qc[tok] = -m;
#pragma unroll
      for (int j = 0; j < EPL; ++j) {
        const int i = lane + 32 * j;
        if (i < E) {
          const float B = x[j] + q + m + (first ? 0.f : qb[row + i]);
          const float v = fminf(B, 0.f);                           // entries above 1 are clipped
          qb[row + i] = B - v;
          L[row + i] = v;
          if (last) A[row + i] = expf(v);
          x[j] = v;
        }
      }
    }
#pragma unroll
    for (int j = 0; j < EPL; ++j) if (lane + 32 * j < E) lse_add(pm[j], ps[j], x[j], 1.f);
  }
#pragma unroll
  for (int j = 0; j < EPL; ++j) if (lane + 32 * j < E) wpart[warp][lane + 32 * j] = make_float2(pm[j], ps[j]);
  __syncthreads();
  for (int i = threadIdx.x; i < E; i += kCapThreads) {
    float m = 0.f, s = 0.f;
    for (int w = 0; w < kCapWarps; ++w) lse_add(m, s, wpart[w][i].x, wpart[w][i].y);
    part_out[((int64_t)g * bpg + blk) * E + i] = make_float2(m, s);
  }
}

__global__ void gather_gate_kernel(const float* __restrict__ S, const int32_t* __restrict__ I, float* __restrict__ G,
                                   int64_t slots_total, int64_t k, int E) {
  for (int64_t s = (int64_t)blockIdx.x * blockDim.x + threadIdx.x; s < slots_total; s += (int64_t)gridDim.x * blockDim.x)
    G[s] = S[(int64_t)I[s] * E + (int)(s / k)];
}

int blocks_per_group(int64_t ng, int groups) {
  int dev = 0, sms = 148;
  cudaGetDevice(&dev);
  cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev);
  int64_t b = sms / groups;
  const int64_t most = (ng + kCapWarps - 1) / kCapWarps;            // at least one token per warp
  if (b > most) b = most;
  return (int)(b < 1 ? 1 : b);
}
// The partials are sized for the largest grid any device could ask for, so the layout does not depend on the device.
constexpr int kCapMaxBlocks = 1024;

size_t align256(size_t b) { return (b + 255) & ~(size_t)255; }

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
  int bpg = blocks_per_group(ng, groups);
  if ((int64_t)bpg * groups > (int64_t)blocks) bpg = (int)(blocks / groups);
  const dim3 grid(bpg, groups);
  const float inv_lambda = 1.f / lambda, log_k = logf((float)kg), log_b = logf((float)b);
  auto round = [&](int phase, int first, int last, const float2* in, float2* out) {
    count_launch();
    if (E <= 32) capped_round_kernel<1><<<grid, kCapThreads, 0, st>>>(S, L, qb, qc, A, in, out, ng, E, inv_lambda, log_k, log_b, phase, first, last);
    else if (E <= 64) capped_round_kernel<2><<<grid, kCapThreads, 0, st>>>(S, L, qb, qc, A, in, out, ng, E, inv_lambda, log_k, log_b, phase, first, last);
    else if (E <= 128) capped_round_kernel<4><<<grid, kCapThreads, 0, st>>>(S, L, qb, qc, A, in, out, ng, E, inv_lambda, log_k, log_b, phase, first, last);
    else capped_round_kernel<8><<<grid, kCapThreads, 0, st>>>(S, L, qb, qc, A, in, out, ng, E, inv_lambda, log_k, log_b, phase, first, last);
  };
  round(0, 0, 0, nullptr, part[0]);
  for (int it = 0; it < iters; ++it) round(1, it == 0, it == iters - 1, part[it & 1], part[(it + 1) & 1]);
  return cudaGetLastError();
}

cudaError_t launch_gather_gate(const float* S, const int32_t* I, float* G, int64_t slots_total, int64_t k, int E,
                               cudaStream_t st) {
  count_launch();
  const int64_t blocks = (slots_total + 255) / 256;
  gather_gate_kernel<<<(unsigned)(blocks > 1184 ? 1184 : blocks), 256, 0, st>>>(S, I, G, slots_total, k, E);
  return cudaGetLastError();
}

}  // namespace ecmoe
