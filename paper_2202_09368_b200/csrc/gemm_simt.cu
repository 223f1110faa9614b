// Plain FMA batched GEMM with arbitrary element strides and the layer's fused epilogues.
// It is the arithmetic of the fp32 path (the 1e-4 tolerance rules out TF32 tensor cores) and the
// fallback for bf16 shapes the tcgen05 kernel does not take.  fp32 accumulation throughout.
#include "internal.h"

namespace ecmoe {

constexpr int BM = 64, BN = 64, BK = 16, TM = 4, TN = 4, NT = 256;

__device__ __forceinline__ float ldv(const float* p, int64_t i) { return p[i]; }
__device__ __forceinline__ float ldv(const bf16* p, int64_t i) { return __bfloat162float(p[i]); }
__device__ __forceinline__ void stv(float* p, int64_t i, float v) { p[i] = v; }
__device__ __forceinline__ void stv(bf16* p, int64_t i, float v) { p[i] = __float2bfloat16(v); }

__device__ __forceinline__ float gelu_fwd(float z, int variant) {
  if (variant == 0) return 0.5f * z * (1.f + erff(z * 0.70710678118654752f));
  const float u = 0.7978845608028654f * (z + 0.044715f * z * z * z);
  return 0.5f * z * (1.f + tanhf(u));
}
__device__ __forceinline__ float gelu_bwd(float z, int variant) {
  if (variant == 0) {
    const float Phi = 0.5f * (1.f + erff(z * 0.70710678118654752f));
    const float phi = 0.3989422804014327f * expf(-0.5f * z * z);
    return Phi + z * phi;
  }
  const float a = 0.7978845608028654f;
  const float th = tanhf(a * (z + 0.044715f * z * z * z));
  return 0.5f * (1.f + th) + 0.5f * z * (1.f - th * th) * a * (1.f + 3.f * 0.044715f * z * z);
}

template <typename TA, typename TB, typename TC>
__global__ void __launch_bounds__(NT) gemm_simt_kernel(GemmArgs g) {
  __shared__ float As[BK][BM + 4];
  __shared__ float Bs[BK][BN + 4];
  const int b = blockIdx.z;
  const TA* A = (const TA*)g.A + (g.a_rows ? 0 : (int64_t)b * g.batch_a);
  const int32_t* arow = g.a_rows ? g.a_rows + (int64_t)b * g.a_rows_batch : nullptr;
  const TB* B = (const TB*)g.B + (int64_t)b * g.batch_b;
  const int m0 = blockIdx.x * BM, n0 = blockIdx.y * BN;     // row tiles on grid.x: M (tokens) is the dimension without a limit
  const int tid = threadIdx.x, tx = tid % 16, ty = tid / 16;
  float acc[TM][TN];
#pragma unroll
  for (int i = 0; i < TM; ++i)
#pragma unroll
    for (int j = 0; j < TN; ++j) acc[i][j] = 0.f;
  const bool a_k_fast = g.sak == 1, b_n_fast = g.sbn == 1;
  int Kb = g.K;
  if (g.k_limit > 0) { const int64_t left = g.k_limit - (int64_t)b * g.K; Kb = (int)(left < g.K ? (left > 0 ? left : 0) : g.K); }
  for (int k0 = 0; k0 < Kb; k0 += BK) {
#pragma unroll
    for (int r = 0; r < BM * BK / NT; ++r) {
      const int idx = tid + r * NT;
      const int mm = a_k_fast ? idx / BK : idx % BM, kk = a_k_fast ? idx % BK : idx / BM;
      const int m = m0 + mm, k = k0 + kk;
      float av = 0.f;
      if (m < g.M && k < Kb) {
        // with a row selection the index along M (or along K) goes through the list first
        int64_t mi = m, ki = k;
        bool ok = true;
        if (arow) {
          const int sel = arow[g.a_rows_k ? k : m];
          ok = idx_ok(sel, 0, g.a_rows_total, g.status);
          if (g.a_rows_k) ki = sel; else mi = sel;
        }
        if (ok) av = ldv(A, mi * g.sam + ki * g.sak);
      }
      As[kk][mm] = av;
    }
#pragma unroll
    for (int r = 0; r < BN * BK / NT; ++r) {
      const int idx = tid + r * NT;
      const int nn = b_n_fast ? idx % BN : idx / BK, kk = b_n_fast ? idx / BN : idx % BK;
      const int n = n0 + nn, k = k0 + kk;
      Bs[kk][nn] = (n < g.N && k < Kb) ? ldv(B, (int64_t)k * g.sbk + (int64_t)n * g.sbn) : 0.f;
    }
    __syncthreads();
#pragma unroll
    for (int kk = 0; kk < BK; ++kk) {
      float a[TM], bb[TN];
#pragma unroll
      for (int i = 0; i < TM; ++i) a[i] = As[kk][ty * TM + i];
#pragma unroll
      for (int j = 0; j < TN; ++j) bb[j] = Bs[kk][tx * TN + j];
#pragma unroll
      for (int i = 0; i < TM; ++i)
#pragma unroll
        for (int j = 0; j < TN; ++j) acc[i][j] = fmaf(a[i], bb[j], acc[i][j]);
    }
    __syncthreads();
  }
  TC* C = (TC*)g.C + (int64_t)b * g.batch_c;
#pragma unroll
  for (int i = 0; i < TM; ++i) {
    const int m = m0 + ty * TM + i;
    if (m >= g.M) continue;
#pragma unroll
    for (int j = 0; j < TN; ++j) {
      const int n = n0 + tx * TN + j;
      if (n >= g.N) continue;
      const int64_t o = (int64_t)m * g.ldc + n;
      float v = acc[i][j];
      if (g.bias) v += g.bias_dtype == 0 ? ((const float*)g.bias)[(int64_t)b * g.N + n] : __bfloat162float(((const bf16*)g.bias)[(int64_t)b * g.N + n]);
      if (g.epi == EPI_GELU) {
        stv((TC*)g.C2 + (int64_t)b * g.batch_c, o, gelu_fwd(v, g.gelu));
      } else if (g.epi == EPI_GELU_GRAD) {
        v *= gelu_bwd(ldv((const TC*)g.Zin + (int64_t)b * g.batch_c, o), g.gelu);
      } else if (g.epi == EPI_ADD_SLOTS) {
        const TC* rows = (const TC*)g.rows;
        int qa = g.row_ptr[m], qb = g.row_ptr[m + 1];
        if (!idx_ok(qa, 0, g.slots_total + 1, n == 0 ? g.status : nullptr) || !idx_ok(qb, qa, g.slots_total + 1, n == 0 ? g.status : nullptr)) qa = qb = 0;
        for (int q = qa; q < qb; ++q) {
          const int sid = g.slots[q];
          if (idx_ok(sid, 0, g.slots_total, n == 0 ? g.status : nullptr)) v += ldv(rows, (int64_t)sid * g.ld_rows + n);
        }
      }
      if (g.C) stv(C, o, v);                    // EPI_GELU without C: only GeLU(acc) is wanted
    }
  }
}

template <typename TA, typename TB>
static void dispatch_c(const GemmArgs& g, dim3 grid, cudaStream_t st) {
  if (g.c_dtype == 0) { count_launch(); gemm_simt_kernel<TA, TB, float><<<grid, NT, 0, st>>>(g); }
  else { count_launch(); gemm_simt_kernel<TA, TB, bf16><<<grid, NT, 0, st>>>(g); }
}

cudaError_t launch_gemm_simt(const GemmArgs& g, cudaStream_t st) {
  const dim3 grid((g.M + BM - 1) / BM, (g.N + BN - 1) / BN, g.batches);
  if (grid.y > 65535u || grid.z > 65535u) return cudaErrorInvalidConfiguration;
  if (g.a_dtype == 0 && g.b_dtype == 0) dispatch_c<float, float>(g, grid, st);
  else if (g.a_dtype == 0) dispatch_c<float, bf16>(g, grid, st);
  else if (g.b_dtype == 0) dispatch_c<bf16, float>(g, grid, st);
  else dispatch_c<bf16, bf16>(g, grid, st);
  return cudaGetLastError();
}

}  // namespace ecmoe
