// Internal declarations shared by the translation units of libecmoe.
// Launch wrappers queue work on the given stream and return the launch status.
#pragma once
#include <cuda_runtime.h>
#include <cuda_bf16.h>
#include <stdint.h>
#include <stddef.h>

namespace ecmoe {

using bf16 = __nv_bfloat16;

constexpr int kTopkChunk = 32;     // experts per histogram CTA column chunk
constexpr int kRadixBits = 10;     // digit width of the radix selection
constexpr int kRadixPasses = 3;    // the 30 significant bits of a score in (0, 1]
constexpr int kCandCap = 512;      // threshold-bucket keys per expert the final sort may choose from
constexpr int kSortTile = 4096;    // 64-bit keys sorted in shared memory by one CTA

// Word 0 of the workspace: status written by kernels (0 = fine, 5 = a bounded wait expired, 6 = an index read from
// I, row_ptr or slots was out of range); word 2 counts such indices.
struct StatusWord { int code; int where; int bad_indices; int pad[61]; };

// Debug build (-DEC_DEBUG): every index read from I, row_ptr or slots is checked against its range before it is used;
// a bad one is recorded in the status word and the access it would have addressed is skipped.  In the normal build
// the check is compiled out.  `status` may be null (the stand-alone shuffle and unshuffle have no workspace): the bad
// access is then skipped without a record.
#ifdef EC_DEBUG
__device__ __forceinline__ bool idx_ok(int64_t i, int64_t lo, int64_t hi, int* status) {
  if (i >= lo && i < hi) return true;
  if (status != nullptr) { atomicExch(status, 6); atomicAdd(status + 2, 1); }
  return false;
}
#else
__device__ __forceinline__ bool idx_ok(int64_t, int64_t, int64_t, int*) { return true; }
#endif

// Per-expert state of the radix selection.
// prefix: key bits decided so far (bits below `shift` are open); k_rem: keys still wanted from the
// threshold bucket; mode: 0 undecided, 1 take the whole bucket, 2 choose k_rem of `cand` candidates,
// 3 ties at the threshold were taken in token order.
struct SelState { unsigned long long prefix; unsigned int k_rem, mode, shift, cand; unsigned int pad[2]; };

// ---- bookkeeping (api.cu) ----------------------------------------------------------------------
// Every kernel launch of the library goes through count_launch(); ec_launch_count() reports the sum.
void count_launch(int n = 1);

// ---- routing (routing.cu) -------------------------------------------------------------------
cudaError_t launch_gate_softmax_simt(int dtype, const void* X, const void* Wg, float* S, int64_t n,
                                     int d, int E, cudaStream_t st);
// scratch layout for the selection is described in routing.cu; bytes needed:
// `groups` independent routing groups of n tokens each (S has groups * n rows); I and G are [E, groups * k],
// group g of an expert at positions g * k .. g * k + k - 1, with global token indices
size_t topk_scratch_bytes(int64_t n, int E, int64_t k, int groups);
cudaError_t launch_topk(const float* S, int64_t n, int E, int64_t k, int groups, int32_t* I, float* G,
                        void* scratch, cudaStream_t st);
// Token-choice contrast (Section 3.1): every token's two best experts (ties: lower expert) into choice [rows, 2];
// then, per expert and group, the requests in token order fill a buffer of k slots: I (-1 = empty), G (0 = empty),
// load and requested [groups, E].
cudaError_t launch_token_top2(const float* S, int64_t rows, int E, int32_t* choice, cudaStream_t st);
cudaError_t launch_token_admit(const float* S, const int32_t* choice, int64_t n, int E, int64_t k, int groups,
                               int32_t* I, float* G, int32_t* load, int32_t* requested, cudaStream_t st);
size_t inverse_scratch_bytes(int64_t n);
// (`status`: the workspace's status word, for the index checks of the debug build; may be null)
cudaError_t launch_inverse_index(const int32_t* I, int64_t n, int64_t slots_total, int32_t* row_ptr,
                                 int32_t* slots, void* scratch, int* status, cudaStream_t st);
cudaError_t launch_gather(int dtype, const void* X, const int32_t* I, void* X_in, int64_t slots_total,
                          int d, int64_t n, int* status, cudaStream_t st);
cudaError_t launch_combine(int dtype, const float* X_e, const float* G, const int32_t* row_ptr,
                           const int32_t* slots, void* X_out, int64_t n, int d, int64_t slots_total, int* status,
                           cudaStream_t st);
// Counts what is wrong with an index structure (every access range-checked): I entries outside [0, n) (or [-1, n) when
// empty slots are allowed) or outside their routing group, row_ptr not starting at 0 / decreasing / not ending at
// the number of filled slots, slots entries out of range, not ascending within a token, or pointing at a slot that
// holds another token.  The count is added to *violations (device).
cudaError_t launch_validate_routing(const int32_t* I, const int32_t* row_ptr, const int32_t* slots, int64_t n, int64_t ng,
                                    int E, int64_t k_total, int64_t kg, int groups, int allow_empty, int* violations,
                                    cudaStream_t st);
// dX_e[s,:] = G[s] * dX_out[I[s],:],  dG[s] = <dX_out[I[s],:], X_e[s,:]>
cudaError_t launch_bwd_combine(int dtype, const void* dX_out, const float* X_e, const float* G,
                               const int32_t* I, void* dX_e, float* dG, int64_t slots_total, int d, int64_t n,
                               int* status, cudaStream_t st);
// dL[t,i] = S[t,i] * (dS[t,i] - sum_i' dS[t,i'] S[t,i']),  dS scattered from dG through the inverse index;
// dL is stored as bf16 when dl_bf16 (operand of the tensor-core dWg / dX products), else fp32
cudaError_t launch_bwd_softmax(const float* S, const float* dG, const int32_t* row_ptr,
                               const int32_t* slots, void* dL, int dl_bf16, int64_t n, int E, int64_t k,
                               int* status, cudaStream_t st);
// out[b, c] = sum over the rows r < min(rows, batch_rows[b]) of A[b, r, c], in ascending r, fp32, cast to dtype
// (gradients of the bias terms: column sums of dZ and dX_e per expert); batch_rows may be null
cudaError_t launch_column_sums(int dtype, const void* A, void* out, int batches, int64_t rows, int cols,
                               const int32_t* batch_rows, cudaStream_t st);
// out[r,c] = sum_p part[p,r,c] in ascending p (fixed order), cast to dtype
cudaError_t launch_reduce_partials(int dtype, const float* part, void* out, int P, int64_t elems,
                                   cudaStream_t st);

// ---- capped expert choice, Section 3.3 (capped.cu) ---------------------------------------------
// A [n, E] (token-major, n = groups * ng): the assignment after `iters` rounds of Dykstra's algorithm with
// Kullback-Leibler projections, per routing group; entries in [0, 1].  E <= 256.
size_t capped_scratch_bytes(int64_t n, int E, int groups);
cudaError_t launch_capped_assignment(const float* S, int64_t ng, int E, int64_t kg, int groups, int b, int iters,
                                     float lambda, float* A, void* scratch, cudaStream_t st);
// G[i, j] = S[I[i, j], i] for I, G of shape [E, k]
cudaError_t launch_gather_gate(const float* S, const int32_t* I, float* G, int64_t slots_total, int64_t k, int E,
                               int64_t n, int* status, cudaStream_t st);

// ---- plain FMA GEMM (gemm_simt.cu) -------------------------------------------------------------
enum Epilogue { EPI_STORE = 0, EPI_GELU = 1, EPI_GELU_GRAD = 2, EPI_ADD_SLOTS = 3 };

struct GemmArgs {
  const void* A; const void* B; void* C;
  int a_dtype, b_dtype, c_dtype;       // ec_dtype values; accumulation is always fp32
  int M, N, K, batches;
  int64_t sam, sak, sbk, sbn, ldc;     // element strides: A[m*sam + k*sak], B[k*sbk + n*sbn], C[m*ldc + n]
  int64_t batch_a, batch_b, batch_c;   // element strides between batches
  int64_t k_limit;                     // if > 0, batch b contracts only min(K, k_limit - b*K) terms (split of a long K)
  int epi, gelu;
  void* C2;                            // EPI_GELU: receives GeLU(acc) (C receives acc, unless C is null)
  const void* Zin;                     // EPI_GELU_GRAD: C = acc * GeLU'(Zin), same layout and dtype as C
  const int32_t* row_ptr; const int32_t* slots; const void* rows; int64_t ld_rows;  // EPI_ADD_SLOTS
  int64_t slots_total; int* status;    // EPI_ADD_SLOTS, debug build: range of the slot ids and where a bad one is recorded
  const void* bias; int bias_dtype;    // not null: bias[b * N + n] is added to the accumulator before the epilogue's function
  // a_rows != null: A is a row selection of one matrix (Eq. 3's X_in = P . X without the copy).  The index along M
  // (a_rows_k = 0) or along K (a_rows_k = 1) is replaced by a_rows[b * a_rows_batch + index], which must lie in
  // [0, a_rows_total); batch_a is unused.
  const int32_t* a_rows; int64_t a_rows_batch, a_rows_total; int a_rows_k;
};
cudaError_t launch_gemm_simt(const GemmArgs& g, cudaStream_t st);

// ---- tcgen05 GEMM (gemm_tc.cu) ---------------------------------------------------------------------
struct TcGemmArgs {
  // C[b][m][n] = sum_k A[b](m,k) * B[b](k,n), bf16 operands, fp32 accumulation in tensor memory.
  const void* A; const void* B;
  int a_mn_major;   // 0: A stored [batch][M][K] (K contiguous); 1: stored [batch][K][M]
  int b_mn_major;   // 0: B stored [batch][N][K] (K contiguous); 1: stored [batch][K][N]
  int M, N, K, batches;
  int64_t lda, ldb; // elements between consecutive rows of the stored matrices
  int64_t batch_a, batch_b;
  int epi, gelu;    // EPI_STORE / EPI_GELU / EPI_GELU_GRAD, or EPI_SOFTMAX below
  void* C; void* C2; const void* Zin; int64_t ldc; int64_t batch_c;   // bf16 outputs (C is fp32 when c_f32);
                                                                      // EPI_GELU with C null writes only C2 = GeLU(acc)
  int c_f32;
  float* S;         // EPI_SOFTMAX: fp32 row softmax of the N columns, [M, N]
  int* status;      // device status word
  // k_split != 0: one matrix product cut along K.  A and B are single matrices (batch strides unused),
  // `batches` is the number of cuts and K the length of one (a multiple of 64); cut b contracts rows
  // b*K .. b*K+K-1 (those at or beyond k_total count as zero) and writes the partial result C[b] (fp32).
  int k_split; int64_t k_total;
  // EPI_ADD_SLOTS (bf16 C, batches == 1): C[m, :] = acc[m, :] + sum over q in [row_ptr[m], row_ptr[m+1]) of
  // rows[slots[q], :] in ascending q, summed in fp32 and rounded once.
  const int32_t* row_ptr; const int32_t* slots; const void* rows; int64_t ld_rows;
  int64_t slots_total;               // EPI_ADD_SLOTS: number of rows of `rows` (the debug build checks the slot ids against it)
  // batch_rows != null: batch b holds only batch_rows[b] meaningful rows along its ragged dimension and zeros after
  // them.  ragged = 1: that dimension is M; row tiles that start at or beyond batch_rows[b] are skipped (never the
  // first one, so rows 0 .. tile-1 of C are always written).  ragged = 2: it is K; k-blocks that start at or beyond
  // batch_rows[b] are skipped (at least one is run).
  const int32_t* batch_rows; int ragged;
  // bias != null (EPI_GELU, or EPI_STORE with fp32 C): bf16 bias[b * N + n] is added to every row of the accumulator
  // before the epilogue's function (the bias terms Eq. 3 leaves out); 16-byte aligned.
  const void* bias;
  // a_rows != null: the shuffle of Eq. 3 read in place.  A's stored rows (its M rows when K-major, its K rows when
  // MN-major) are rows of ONE matrix [a_rows_total, lda] at A, chosen through an index list: stored row r of batch b
  // is matrix row a_rows[b * a_rows_batch + r] (every entry in [0, a_rows_total)).  batch_a is unused; not with
  // k_split or batch_rows.
  const int32_t* a_rows; int64_t a_rows_batch, a_rows_total;
};
constexpr int EPI_SOFTMAX = 4;
bool tc_gemm_supported(const TcGemmArgs& g);
cudaError_t launch_gemm_tc(const TcGemmArgs& g, cudaStream_t st);

}  // namespace ecmoe
