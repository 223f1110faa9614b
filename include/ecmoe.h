/*
 * ecmoe.h - C ABI of the expert-choice (EC) mixture-of-experts feed-forward layer
 * for NVIDIA B200 (sm_100a).
 *
 * The layer is the one of "Mixture-of-Experts with Expert Choice Routing"
 * (arXiv 2202.09368), Section 3.2.  Notation follows the paper: n tokens in the
 * routed group, d model width, d' hidden width of an expert, e experts, capacity
 * factor c, k = n*c/e tokens per expert (Eq. 1).  A "slot" is one (expert i,
 * position j) pair; its flat id is i*k + j and there are e*k of them.
 *
 * Routing groups.  The paper routes one group of n tokens (Section 3.2) and names, under
 * Limitations, routing several groups independently as the way to use the method where a
 * token must not compete with all others (for example, tokens of one sequence spread over
 * groups).  cfg->groups = g > 1 does that: X holds g*n rows, group r being rows r*n ..
 * r*n + n - 1 (how tokens are assigned to groups is the caller's arrangement of X); every
 * expert takes the top k = n*c/e tokens of each group, so it serves g*k slots.  In every
 * shape below read then n as g*n (rows of X, S, X_out, row_ptr) and k as g*k (row length of
 * I and G, slots per expert), with an expert's slots ordered by group and, inside a group,
 * as for one group; token indices are global row numbers of X.  g = 1 is the paper's layer.
 *
 * Conventions for every entry point unless it says otherwise
 *  - Tensor arguments are DEVICE pointers owned by the caller, dense row-major,
 *    16-byte aligned.  The library never allocates, frees or keeps device memory.
 *  - Work is queued on `cuda_stream` (a cudaStream_t passed as void*; NULL is the
 *    legacy default stream) and the call returns without synchronising; results
 *    are valid once the caller has synchronised that stream.
 *  - `ws` is scratch of at least ec_workspace_bytes(cfg) bytes, 256-byte aligned;
 *    its contents are undefined after a call.  Two calls that overlap on the GPU
 *    must not share a workspace.
 *  - Errors are return codes.  Arguments are checked on the host before anything
 *    is launched; nothing is launched when the code is not EC_OK.
 *  - X, Wg, W1, W2, X_out, dX_out and all gradients have the element type
 *    cfg->dtype; S, G and X_e are always fp32 and index outputs are int32.
 *  - Restrictions (EC_ERR_UNSUPPORTED otherwise): d_model and d_ff rows must be a
 *    multiple of 16 bytes long and d_model, d_ff <= 2^22 - 64; groups*n < 2^31; 1 <= E <= 256;
 *    E*groups*k < 2^31; 1 <= groups <= 65535.
 *  - Host threads: calls that use different workspaces (and different saved blobs) may run
 *    concurrently from different host threads; the library keeps no per-call state outside
 *    the buffers it is handed.  The exceptions say so in their own comments (ec_route_static's
 *    shared array, the process-wide ec_profile_* and ec_launch_count).
 */
#ifndef ECMOE_H_
#define ECMOE_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef enum {
  EC_OK = 0,
  EC_ERR_INVALID_ARG = 1, /* null pointer, misaligned pointer, k outside [1, n], bad enum        */
  EC_ERR_UNSUPPORTED = 2, /* a documented restriction is violated                                */
  EC_ERR_WORKSPACE = 3,   /* ws_bytes or saved_bytes smaller than required                       */
  EC_ERR_CUDA = 4,        /* a CUDA runtime or driver call failed (launch, tensor-map encode)    */
  EC_ERR_TIMEOUT = 5,     /* a bounded device-side wait expired (reported by ec_read_status)     */
  EC_ERR_INDEX = 6        /* debug build only: an index read from I, row_ptr or slots was out of
                             range; the access was skipped (reported by ec_read_status)          */
} ec_status;

typedef enum { EC_F32 = 0, EC_BF16 = 1 } ec_dtype;
typedef enum { EC_GELU_ERF = 0, EC_GELU_TANH = 1 } ec_gelu;
/* Who chooses: EC_ROUTER_EXPERT_CHOICE is the paper's method (Section 3.2).  EC_ROUTER_TOKEN_TOP2 is the conventional
 * routing Section 3.1 contrasts it with, provided as a synthetic contrast workload on the same layer: every token picks
 * its two highest-scoring experts (equal scores: the lower expert), an expert's buffer holds k = n*c/e tokens (Eq. 1's
 * formula read as the buffer size), takes requests in token order and drops what does not fit.  Slots are then filled
 * in order of arrival, I holds -1 and G holds 0 in empty slots, tokens have 0, 1 or 2 experts, and everything after
 * the routing (Eq. 3-4, the backward pass with the choices held constant) is the same code on those slots; the
 * tensor-core GEMMs skip the tiles and k-blocks that hold only empty slots (with groups = 1). */
typedef enum { EC_ROUTER_EXPERT_CHOICE = 0, EC_ROUTER_TOKEN_TOP2 = 1 } ec_router;

/* One layer call.  Plain data, passed by pointer, never retained. */
typedef struct {
  int64_t n;       /* tokens in the group (Section 3.2: batch size x sequence length) */
  int32_t d_model; /* d                                                               */
  int32_t d_ff;    /* d'                                                              */
  int32_t E;       /* number of experts e                                             */
  int32_t groups;  /* independent routing groups of n tokens each, >= 1 (see above)       */
  double c;        /* capacity factor (Eq. 1)                                         */
  int32_t dtype;   /* ec_dtype                                                        */
  int32_t gelu;    /* ec_gelu                                                         */
  /* Section 3.3, expert choice with at most cap_b experts per token; cap_b = 0 switches it off. */
  int32_t cap_b;     /* b: bound on the column sums of A; needs E*k <= n*b                      */
  int32_t cap_iters; /* rounds of Dykstra's algorithm (the paper: at most 100), >= 1            */
  double cap_lambda; /* weight of the entropy term (the paper: 0.001), > 0                      */
  int32_t router;    /* ec_router; the token-choice contrast needs cap_b = 0 and E >= 2         */
  /* 1: Eq. 3's shuffle X_in = P . X is never written.  GEMM-1 and the dW1 product read the chosen rows of X in place
   * through I (row-indexed TMA loads on the tensor-core path), the blob of ec_saved_bytes is smaller by E*k*d elements
   * and ec_saved_view reports X_in = NULL; every result is bit-identical to fuse_gather = 0.  It trades time for that
   * memory: the rows are fetched again for every column tile, which is slower than gathering once.  Expert choice
   * only (empty slots have no row to read).  0: the rows are gathered once into X_in.                               */
  int32_t fuse_gather;
} ec_config;

/* Views into the forward->backward blob (device pointers), for inspection and tests. */
typedef struct {
  float* S;         /* [n, E]     gate scores (Eq. 2)                                  */
  int32_t* I;       /* [E, k]     token chosen for each slot                           */
  float* G;         /* [E, k]     gate weight of each slot, G[i,j] = S[I[i,j], i]      */
  int32_t* row_ptr; /* [n+1]      token -> range in `slots`                            */
  int32_t* slots;   /* [E*k]      flat slot ids of each token, ascending               */
  void* X_in;       /* [E, k, d]  gathered expert inputs (Eq. 3); NULL with fuse_gather  */
  void* Z;          /* [E, k, d'] X_in[i] . W1[i]                                      */
  void* H;          /* [E, k, d'] GeLU(Z)                                              */
  float* X_e;       /* [E, k, d]  expert outputs H[i] . W2[i]^T, fp32 on both paths    */
  int32_t* load;      /* [groups, E] slots filled per expert (EC_ROUTER_TOKEN_TOP2 only, else NULL)   */
  int32_t* requested; /* [groups, E] tokens that asked for the expert, before dropping (same)         */
} ec_saved_ptrs;

/* Eq. 1: k = floor(n*c/E), per routing group.  Returns -1 when cfg is NULL or k falls outside [1, n]. */
int64_t ec_capacity(const ec_config* cfg);

/* Bytes of scratch every call below needs (the maximum over the three).  0 on a bad cfg. */
size_t ec_workspace_bytes(const ec_config* cfg);

/* Bytes of scratch a forward-only call of ec_moe_forward (saved == NULL) needs: the routing scratch plus every
 * intermediate of Eq. 2-3 except Z.  0 on a bad cfg. */
size_t ec_forward_only_workspace_bytes(const ec_config* cfg);

/* Bytes of the blob ec_moe_forward fills for ec_moe_backward.  0 on a bad cfg. */
size_t ec_saved_bytes(const ec_config* cfg);

/* Computes the addresses of the blob's parts.  Host-only arithmetic; `saved` is not touched. */
ec_status ec_saved_view(const ec_config* cfg, void* saved, ec_saved_ptrs* out);

/*
 * Routing, Eq. 1-2: S = Softmax(X . Wg) over the E experts of each token, then for
 * every expert the k largest entries of its column of S.  Ties go to the lower
 * token index; each expert's slots are listed by descending score (equal scores
 * by ascending token), which makes I and G unique.  Also emits the index form of
 * P = Onehot(I) read by token: slots[row_ptr[t] .. row_ptr[t+1]) are the flat
 * slot ids that hold token t, ascending (so ascending expert).
 *   X [n, d], Wg [d, E] in;  S [n, E], I [E, k], G [E, k], row_ptr [n+1], slots [E*k] out.
 * On the bf16 path logits are accumulated in fp32 and the softmax and the
 * comparison run on fp32 values.
 */
ec_status ec_route(const ec_config* cfg, const void* X, const void* Wg, float* S, int32_t* I,
                   float* G, int32_t* row_ptr, int32_t* slots, void* ws, size_t ws_bytes,
                   void* cuda_stream);

/*
 * The token-choice contrast routing (see ec_router) on its own; cfg->router must be EC_ROUTER_TOKEN_TOP2 (ec_route and
 * ec_route_static refuse such a cfg with EC_ERR_INVALID_ARG: they have nowhere to put the loads).  Outputs as for
 * ec_route, with -1 / 0 in the empty slots of I / G and only the first row_ptr[n] entries of `slots` written, plus
 * load and requested, [groups, E] int32 each: slots filled per expert and tokens that asked for it.  max(requested) / k
 * is how far the fullest expert is over its buffer (Section 3.1's over-capacity ratio, plus one).
 */
ec_status ec_route_token_choice(const ec_config* cfg, const void* X, const void* Wg, float* S, int32_t* I,
                                float* G, int32_t* row_ptr, int32_t* slots, int32_t* load,
                                int32_t* requested, void* ws, size_t ws_bytes, void* cuda_stream);

/*
 * Section 3.3 on its own: the assignment A of
 *     max <S^T, A> + cap_lambda * H(A)   s.t.  rows sum to k, columns sum to at most cap_b, 0 <= A <= 1
 * after cap_iters rounds of Dykstra's algorithm with Kullback-Leibler projections (one round: rows, then
 * columns, then the box, each applied to the iterate times that set's correction factor), started from
 * exp(S^T / cap_lambda), computed on log A in fp32.  S [n, E] in, A [n, E] out (token-major like S: A[t, i] is
 * the section's A[i, t]), entries in [0, 1]; routing groups are solved independently.  With cfg->cap_b > 0
 * ec_route, ec_route_static and ec_moe_forward run this after the gate and take I = TopK(A, k) (same order and
 * tie rule as Eq. 2) with G[i, j] = S[I[i, j], i]; everything downstream, the backward pass included, is
 * unchanged (I is a constant there).  This entry point exists to inspect A; it needs cfg->cap_b > 0
 * (EC_ERR_INVALID_ARG otherwise) and the workspace of ec_workspace_bytes.  At cap_lambda = 0.001 the iteration
 * advances about log(k / current row sum) per round in log A, so whether the stated 100 rounds reach rows that
 * sum to k depends on how the scores are spread; cap_iters is the caller's to raise.
 */
ec_status ec_capped_assignment(const ec_config* cfg, const float* S, float* A, void* ws, size_t ws_bytes,
                               void* cuda_stream);

/*
 * The shuffle of Eq. 3 on its own: X_in[i, j, :] = X[I[i, j], :] (X_in = P . X with P = Onehot(I)),
 * a row gather.  X [n, d] and I [E, k] in, X_in [E, k, d] out, both of cfg->dtype.  Entries of I
 * must lie in [0, n).  No workspace.
 */
ec_status ec_shuffle(const ec_config* cfg, const void* X, const int32_t* I, void* X_in,
                     void* cuda_stream);

/*
 * The unshuffle of Eq. 4 on its own: X_out[t, :] = sum over the slots s = (i, j) that hold token t of
 * G[s] * X_e[s, :], slots in ascending order, accumulated in fp32 and rounded once; rows of
 * tokens without a slot are zero.  X_e [E, k, d] fp32, G [E, k] fp32 and the token -> slot index
 * (row_ptr [n+1], slots [E*k], as ec_route writes them) in, X_out [n, d] of cfg->dtype out.
 * No workspace, no atomics: the result does not depend on scheduling.
 */
ec_status ec_unshuffle(const ec_config* cfg, const float* X_e, const float* G, const int32_t* row_ptr,
                       const int32_t* slots, void* X_out, void* cuda_stream);

/*
 * Routing for callers that cannot allocate device memory.  The paper has no counterpart:
 * this is ec_route with the workspace argument taken away.
 *
 * Who needs it: code that is handed its input and output buffers by someone else and
 * has no allocator of its own to ask for scratch, for example a plug-in running inside
 * a host framework that owns all device memory, a real-time or serving loop in which
 * cudaMalloc is forbidden because it synchronises the device and can fail or stall at
 * an arbitrary moment, or a process whose memory budget was fixed at start-up.  Such a
 * caller still passes X, Wg and the five outputs exactly as for ec_route; the scratch
 * (status word, selection histograms and keys, inverse-index cursor) comes from a fixed
 * array of EC_ROUTE_STATIC_SCRATCH_BYTES bytes that is part of the library's device
 * image.  Every GPU on which the library is used holds that array from the moment the
 * library's device code is loaded there until the process exits.
 *
 * Limits and behaviour
 *  - A configuration whose routing scratch (ec_route_static_bytes(cfg)) exceeds
 *    EC_ROUTE_STATIC_SCRATCH_BYTES is refused with EC_ERR_WORKSPACE and nothing is
 *    launched; use ec_route with a workspace of your own for it.  8 MiB covers, for
 *    instance, n = 262144 with E = 8 .. 256 at c = 2.
 *  - The call itself makes no allocation: no cudaMalloc / cudaFree, no allocating
 *    library routine.  The first call on each device looks up the array's device address
 *    (once, with that device current, under a lock); make that first call outside any
 *    stream capture.  Later calls on that device only queue work on `cuda_stream`.
 *  - All calls on one device share the one array and it keeps the previous call's
 *    contents; everything that must start at zero is cleared on `cuda_stream` at the
 *    start of each call.  Two calls that can overlap on the GPU (different streams
 *    without an ordering between them, or different host threads doing so) race on the
 *    array and give undefined results: order them, or use ec_route with separate
 *    workspaces.  There is no status word to read back afterwards; a caller that needs
 *    ec_read_status uses ec_route.
 *  - Results are those of ec_route on the same inputs, bit for bit.
 */
#define EC_ROUTE_STATIC_SCRATCH_BYTES (8u << 20)
size_t ec_route_static_bytes(const ec_config* cfg); /* scratch this cfg needs; 0 on a bad cfg */
ec_status ec_route_static(const ec_config* cfg, const void* X, const void* Wg, float* S,
                          int32_t* I, float* G, int32_t* row_ptr, int32_t* slots,
                          void* cuda_stream);

/*
 * Forward, Eq. 2-4: routing as above, X_in = P . X (gather), X_e[i] =
 * GeLU(X_in[i] . W1[i]) . W2[i]^T for every expert, and X_out[t, :] = sum over the
 * slots (i, j) holding t of G[i, j] * X_e[i, j, :], experts in ascending order, in
 * fp32, rounded once.  Rows of tokens that no expert chose are zero.
 *   W1, W2 [E, d, d'] (W2 is applied transposed);  X_out [n, d] out.
 * b1 [E, d'] and b2 [E, d] (cfg->dtype, 16-byte aligned) are the bias terms the paper leaves out of Eq. 3 "for
 * brevity": X_e[i] = GeLU(X_in[i] . W1[i] + b1[i]) . W2[i]^T + b2[i].  Either may be NULL (no such term: the equation
 * as printed).
 * `saved` (ec_saved_bytes(cfg) bytes, 256-byte aligned) receives what the backward
 * pass needs (the intermediates live there).  Forward only (inference): pass saved = NULL
 * and saved_bytes = 0; the intermediates then live in `ws`, which must hold
 * ec_forward_only_workspace_bytes(cfg) bytes, and Z = X_in . W1, which only the backward
 * pass reads, is not written at all.  X_out is the same, bit for bit.
 */
ec_status ec_moe_forward(const ec_config* cfg, const void* X, const void* Wg, const void* W1,
                         const void* W2, const void* b1, const void* b2, void* X_out, void* saved,
                         size_t saved_bytes, void* ws, size_t ws_bytes, void* cuda_stream);

/*
 * Backward of Eq. 2-4 (the paper trains the gate, Section 3.4, and leaves the
 * derivative to automatic differentiation): gradients of <dX_out, X_out> with I held
 * constant, so the gate receives gradient through G only.
 *   dX_out [n, d] in, `saved` as filled by ec_moe_forward with the same cfg and inputs;
 *   dX [n, d], dWg [d, E], dW1, dW2 [E, d, d'] out, overwritten (not accumulated);
 *   db1 [E, d'], db2 [E, d] out, the gradients of the bias terms (sums of dZ and of dX_e over an expert's slots,
 *   in slot order, fp32, rounded once); either may be NULL (not wanted).  The biases themselves are not needed here:
 *   the saved Z already contains b1.
 */
ec_status ec_moe_backward(const ec_config* cfg, const void* X, const void* Wg, const void* W1,
                          const void* W2, const void* dX_out, const void* saved,
                          size_t saved_bytes, void* dX, void* dWg, void* dW1, void* dW2, void* db1,
                          void* db2, void* ws, size_t ws_bytes, void* cuda_stream);

/*
 * One expert-batched product of Eq. 3 or of its backward on its own (benchmarks time the kernels apart from the layer
 * with it; ec_moe_forward / ec_moe_backward run the same kernels).  k = ec_capacity(cfg) * groups rows per expert,
 * d = d_model, d' = d_ff, all operands and the result of cfg->dtype, dense, [E, rows, columns]:
 *   EC_GEMM_XW1   C[i] = A[i] . B[i]        A [E, k, d],  B [E, d, d'] (W1's layout)       -> C [E, k, d']
 *   EC_GEMM_HW2T  C[i] = A[i] . B[i]^T      A [E, k, d'], B [E, d, d'] (W2's layout)       -> C [E, k, d]
 *   EC_GEMM_ATB   C[i] = A[i]^T . B[i]      A [E, k, d],  B [E, k, d'] (the weight gradients) -> C [E, d, d']
 * fp32 accumulation, one rounding to cfg->dtype.  `ws` as for the other calls (only its status word is used).
 */
typedef enum { EC_GEMM_XW1 = 0, EC_GEMM_HW2T = 1, EC_GEMM_ATB = 2 } ec_gemm_kind;
ec_status ec_expert_gemm(const ec_config* cfg, int kind, const void* A, const void* B, void* C, void* ws,
                         size_t ws_bytes, void* cuda_stream);

/*
 * Checks an index structure as ec_route / ec_route_token_choice produce it (the paper has no counterpart; for callers
 * that build or modify I, row_ptr, slots themselves before ec_shuffle / ec_unshuffle, and for debugging): every entry
 * of I [E, k] is a token of the slot's own routing group (or -1 with the token-choice router), row_ptr [n+1] starts at
 * 0, never decreases and ends at the number of filled slots, and every token's list in `slots` is ascending, in range
 * and points at slots that hold that token.  Any contents are safe to pass: every access is range-checked.  Writes
 * the number of violations found to *violations (host memory) and synchronises `cuda_stream`.
 */
ec_status ec_validate_routing(const ec_config* cfg, const int32_t* I, const int32_t* row_ptr,
                              const int32_t* slots, int64_t* violations, void* ws, size_t ws_bytes,
                              void* cuda_stream);

/* 1 if this library was built with -DEC_DEBUG: every kernel then range-checks each index it reads from I, row_ptr
 * or slots before using it, skips the access when it is out of range and records EC_ERR_INDEX in the status word
 * (ec_read_status).  The normal build compiles these checks out. */
int ec_debug_build(void);

/* Views into the workspace as ec_moe_backward leaves it (device pointers; valid until the next call that uses the
 * workspace), for inspection and tests: the intermediates of the chain rule through Eq. 4, 3 and 2.  Rows of dZ and
 * dX_in that belong to empty slots (token-choice router) are unspecified. */
typedef struct {
  void* dX_e;         /* [E, k, d]  G[i,j] * dX_out[I[i,j], :], cfg->dtype                       */
  float* dG;          /* [E, k]     <dX_out[I[i,j], :], X_e[i,j,:]>                              */
  void* dZ;           /* [E, k, d'] (dX_e[i] . W2[i]) * GeLU'(Z), cfg->dtype                     */
  void* dX_in;        /* [E, k, d]  dZ[i] . W1[i]^T, cfg->dtype                                  */
  void* dL;           /* [n, E]     gradient of the gate logits; bf16 if dL_is_bf16, else fp32   */
  int32_t dL_is_bf16; /* 1 when the two gate-gradient products run on the tensor cores           */
} ec_backward_ptrs;
ec_status ec_backward_view(const ec_config* cfg, void* ws, ec_backward_ptrs* out);

/*
 * Synchronises `cuda_stream` and reads the status word the kernels of the last call
 * on `ws` left there: EC_OK, or EC_ERR_TIMEOUT when a bounded wait inside a kernel
 * gave up (the outputs of that call are then undefined), or EC_ERR_INDEX (debug build)
 * when an index was out of range, or EC_ERR_CUDA when the stream reports an error.
 */
ec_status ec_read_status(const void* ws, void* cuda_stream);

/* Static, NUL-terminated description of a status code. */
const char* ec_status_string(ec_status s);

/* 1 if the bf16 path of this cfg runs its expert GEMMs on the tcgen05 tensor-core
 * kernels, 0 if it falls back to the plain FMA kernels (fp32 path, odd shapes). */
int ec_uses_tensor_cores(const ec_config* cfg);

/* Number of CUDA kernels this library has launched in this process so far (all calls, all
 * streams).  The paper has no counterpart; benchmarks use the difference across a timed region. */
long long ec_launch_count(void);

/*
 * Per-stage device timing, for benchmarks (no counterpart in the paper).  After
 * ec_profile_enable(1), each call of ec_route / ec_moe_forward / ec_moe_backward records a CUDA
 * event on its stream after every stage (gate, top-k, inverse index, gather, the GEMMs, combine,
 * ...).  The events of the last routing / forward call and of the last backward call are kept
 * apart, so a forward and a backward queued back to back can both be read afterwards.
 * ec_profile_read waits for those calls' final events and writes up to max_stages elapsed times
 * (milliseconds) and static stage names, forward stages first, then backward; it returns the
 * number of stages written (what it returned is not returned again), 0 when profiling is off or
 * nothing was recorded, -1 on a CUDA error.  The state is global to the process: use it from one
 * thread, one call of each kind at a time.  Off by default.
 */
void ec_profile_enable(int on);
int ec_profile_read(float* ms, const char** names, int max_stages);

#ifdef __cplusplus
}
#endif
#endif /* ECMOE_H_ */
