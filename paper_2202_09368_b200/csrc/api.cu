// C ABI of the expert-choice MoE layer: argument checks, workspace carving and the sequence of
// kernel launches for routing (Eq. 1-2), forward (Eq. 2-4) and backward.
#include "../../include/ecmoe.h"
#include "internal.h"

#include <math.h>
#include <string.h>
#include <atomic>
#include <mutex>

using namespace ecmoe;

namespace {

constexpr size_t kAlign = 256;
inline size_t up(size_t b) { return (b + kAlign - 1) & ~(kAlign - 1); }
inline size_t esize(int dtype) { return dtype == EC_F32 ? 4 : 2; }

// n: all tokens of the call (groups * tokens per group), k: slots per expert (groups * k per group),
// slots = E * k; ng, kg: the per-group values Eq. 1 is about.
struct Dims { int64_t n, k, slots, ng, kg; int d, dff, E, groups; int dtype, gelu; size_t eb;
              int cap_b, cap_iters; double cap_lambda; int router, fuse; };

ec_status check_cfg(const ec_config* c, Dims* D) {
  if (!c) return EC_ERR_INVALID_ARG;
  if (c->dtype != EC_F32 && c->dtype != EC_BF16) return EC_ERR_INVALID_ARG;
  if (c->gelu != EC_GELU_ERF && c->gelu != EC_GELU_TANH) return EC_ERR_INVALID_ARG;
  if (c->n < 1 || c->d_model < 1 || c->d_ff < 1 || c->E < 1 || !(c->c > 0.0)) return EC_ERR_INVALID_ARG;
  if (c->groups < 1) return EC_ERR_INVALID_ARG;
  if (c->n * c->groups >= ((int64_t)1 << 31) || c->E > 256 || c->groups > 65535) return EC_ERR_UNSUPPORTED;
  const size_t eb = esize(c->dtype);
  if ((c->d_model * eb) % 16 || (c->d_ff * eb) % 16) return EC_ERR_UNSUPPORTED;
  if (c->d_model > (1 << 22) - 64 || c->d_ff > (1 << 22) - 64) return EC_ERR_UNSUPPORTED;   // column tiles of the FMA kernels sit on grid.y
  const int64_t k = ec_capacity(c);
  if (k < 1) return EC_ERR_INVALID_ARG;
  if ((int64_t)c->E * k * c->groups >= ((int64_t)1 << 31)) return EC_ERR_UNSUPPORTED;
  if (c->cap_b < 0) return EC_ERR_INVALID_ARG;
  if (c->cap_b > 0) {
    if (c->cap_iters < 1 || !(c->cap_lambda > 0.0)) return EC_ERR_INVALID_ARG;
    if ((int64_t)c->E * k > c->n * (int64_t)c->cap_b) return EC_ERR_INVALID_ARG;     // E*k slots cannot fit under the cap
  }
  if (c->router != EC_ROUTER_EXPERT_CHOICE && c->router != EC_ROUTER_TOKEN_TOP2) return EC_ERR_INVALID_ARG;
  if (c->router == EC_ROUTER_TOKEN_TOP2 && (c->cap_b != 0 || c->E < 2)) return EC_ERR_INVALID_ARG;
  if (c->fuse_gather != 0 && c->fuse_gather != 1) return EC_ERR_INVALID_ARG;
  if (c->fuse_gather && c->router != EC_ROUTER_EXPERT_CHOICE) return EC_ERR_INVALID_ARG;   // empty slots have no row of X to read
  if (D) { D->router = c->router; D->fuse = c->fuse_gather; D->ng = c->n; D->kg = k; D->groups = c->groups; D->n = c->n * c->groups; D->k = k * c->groups;
           D->slots = (int64_t)c->E * D->k; D->d = c->d_model; D->dff = c->d_ff;
           D->E = c->E; D->dtype = c->dtype; D->gelu = c->gelu; D->eb = eb;
           D->cap_b = c->cap_b; D->cap_iters = c->cap_iters; D->cap_lambda = c->cap_lambda; }
  return EC_OK;
}

struct SavedLayout { size_t S, I, G, row_ptr, slots, X_in, Z, H, X_e, load, requested, total; };
// with_z = false: the layout of the same tensors without Z (forward-only calls keep them in the workspace)
SavedLayout saved_layout(const Dims& D, bool with_z = true) {
  SavedLayout L; size_t o = 0;
  auto take = [&](size_t b) { size_t r = o; o += up(b); return r; };
  L.S = take((size_t)D.n * D.E * 4);
  L.I = take((size_t)D.slots * 4);
  L.G = take((size_t)D.slots * 4);
  L.row_ptr = take((size_t)(D.n + 1) * 4);
  L.slots = take((size_t)D.slots * 4);
  L.X_in = take(D.fuse ? 0 : (size_t)D.slots * D.d * D.eb);       // with fuse_gather the rows of X are read in place
  L.Z = take(with_z ? (size_t)D.slots * D.dff * D.eb : 0);
  L.H = take((size_t)D.slots * D.dff * D.eb);
  L.X_e = take((size_t)D.slots * D.d * 4);          // fp32 on both paths
  L.load = take(D.router ? (size_t)D.groups * D.E * 4 : 0);         // token-choice contrast only
  L.requested = take(D.router ? (size_t)D.groups * D.E * 4 : 0);
  L.total = o;
  return L;
}

// Number of fixed cuts of the token axis in dWg = X^T . dL: enough (row tile, cut) pairs for about two
// waves of CTAs, at least 512 tokens per cut, at most 32 cuts.  Depends on the shape only, so the
// summation order, and with it the result, is the same on every run.
int dwg_splits(const Dims& D) {
  const int64_t tiles_m = (D.d + 127) / 128;
  int64_t p = 296 / tiles_m;
  if (p > D.n / 512) p = D.n / 512;
  return (int)(p < 1 ? 1 : (p > 32 ? 32 : p));
}

struct WsLayout { size_t status, topk, inverse, cap_A, capped, choice, fwd_end, dX_e, dG, dZ, dX_in, dL, dWg_part, total; };
WsLayout ws_layout(const Dims& D) {
  WsLayout L; size_t o = 0;
  auto take = [&](size_t b) { size_t r = o; o += up(b); return r; };
  L.status = take(sizeof(StatusWord));
  const size_t base = o;
  L.topk = take(topk_scratch_bytes(D.ng, D.E, D.kg, D.groups));
  L.inverse = take(inverse_scratch_bytes(D.n));
  L.cap_A = take(D.cap_b ? (size_t)D.n * D.E * 4 : 0);
  L.capped = take(D.cap_b ? capped_scratch_bytes(D.n, D.E, D.groups) : 0);
  L.choice = take(D.router ? (size_t)D.n * 2 * 4 : 0);              // every token's two experts (token-choice contrast)
  const size_t fwd_end = o;
  L.fwd_end = fwd_end;
  o = base;                                   // the backward pass reuses the same region
  L.dX_e = take((size_t)D.slots * D.d * D.eb);
  L.dG = take((size_t)D.slots * 4);
  L.dZ = take((size_t)D.slots * D.dff * D.eb);
  L.dX_in = take((size_t)D.slots * D.d * D.eb);
  L.dL = take((size_t)D.n * D.E * 4);
  L.dWg_part = take((size_t)dwg_splits(D) * D.d * D.E * 4);
  L.total = o > fwd_end ? o : fwd_end;
  return L;
}

inline bool misaligned(const void* p, size_t a) { return ((uintptr_t)p & (a - 1)) != 0; }

#define EC_CUDA(x) do { if ((x) != cudaSuccess) return EC_ERR_CUDA; } while (0)

// Optional per-stage timing (ec_profile_enable): an event is recorded on the call's stream after
// each stage.  Two sets of events, one for routing / forward calls and one for backward calls, so
// that a forward + backward pair queued back to back can be read afterwards without a
// synchronisation in between.  Host state only; off by default and then free of cost.
constexpr int kMaxStages = 20;
struct Profile {
  cudaEvent_t ev[kMaxStages + 1];
  bool created = false;
  int count = 0;                       // stages recorded by the last call of this kind
  const char* names[kMaxStages];
};
bool g_prof_enabled = false;
Profile g_prof[2];
int g_prof_cur = 0;
std::atomic<long long> g_launches{0};

void prof_begin(cudaStream_t st, int kind) {
  if (!g_prof_enabled) return;
  Profile& P = g_prof[kind];
  g_prof_cur = kind;
  if (!P.created) { for (auto& e : P.ev) cudaEventCreate(&e); P.created = true; }
  P.count = 0;
  cudaEventRecord(P.ev[0], st);
}
void prof_mark(const char* name, cudaStream_t st) {
  Profile& P = g_prof[g_prof_cur];
  if (!g_prof_enabled || P.count >= kMaxStages) return;
  P.names[P.count] = name;
  cudaEventRecord(P.ev[++P.count], st);
}

// One expert-batched GEMM: tensor cores when the shape allows, FMA otherwise.
struct BatchedGemm {
  const void* A; int a_mn; int64_t lda, batch_a;     // a_mn = 0: A stored [M][K]; 1: stored [K][M]
  const void* B; int b_mn; int64_t ldb, batch_b;     // b_mn = 0: B stored [N][K]; 1: stored [K][N]
  void* C; int64_t ldc, batch_c;
  int M, N, K, batches, epi;
  void* C2; const void* Zin;
  int c_f32;                                         // C is fp32 regardless of the path's dtype
  const int32_t* batch_rows; int ragged;             // see TcGemmArgs: meaningful rows per batch along M (1) or K (2)
  const void* bias;                                  // [batches, N] of the path's dtype, added to the accumulator (Eq. 3's omitted bias terms)
  // A's stored rows are rows of the matrix at A (a_rows_total rows, pitch lda) picked through a_rows (Eq. 3's
  // X_in = P . X read in place): row r of batch b is matrix row a_rows[b * a_rows_batch + r]
  const int32_t* a_rows; int64_t a_rows_batch, a_rows_total;
};

ec_status run_gemm(const Dims& D, const BatchedGemm& b, int* status_word, cudaStream_t st) {
  if (D.dtype == EC_BF16) {
    TcGemmArgs t; memset(&t, 0, sizeof(t));
    t.A = b.A; t.B = b.B; t.a_mn_major = b.a_mn; t.b_mn_major = b.b_mn;
    t.M = b.M; t.N = b.N; t.K = b.K; t.batches = b.batches;
    t.lda = b.lda; t.ldb = b.ldb; t.batch_a = b.batch_a; t.batch_b = b.batch_b;
    t.epi = b.epi; t.gelu = D.gelu; t.C = b.C; t.C2 = b.C2; t.Zin = b.Zin; t.ldc = b.ldc; t.batch_c = b.batch_c; t.c_f32 = b.c_f32;
    t.status = status_word;
    t.batch_rows = b.batch_rows; t.ragged = b.ragged; t.bias = b.bias;
    t.a_rows = b.a_rows; t.a_rows_batch = b.a_rows_batch; t.a_rows_total = b.a_rows_total;
    if (tc_gemm_supported(t)) { EC_CUDA(launch_gemm_tc(t, st)); return EC_OK; }
  }
  GemmArgs g; memset(&g, 0, sizeof(g));
  g.A = b.A; g.B = b.B; g.C = b.C; g.a_dtype = g.b_dtype = g.c_dtype = D.dtype;
  if (b.c_f32) g.c_dtype = EC_F32;
  g.M = b.M; g.N = b.N; g.K = b.K; g.batches = b.batches;
  g.sam = b.a_mn ? 1 : b.lda; g.sak = b.a_mn ? b.lda : 1;
  g.sbk = b.b_mn ? b.ldb : 1; g.sbn = b.b_mn ? 1 : b.ldb;
  g.ldc = b.ldc; g.batch_a = b.batch_a; g.batch_b = b.batch_b; g.batch_c = b.batch_c;
  g.epi = b.epi; g.gelu = D.gelu; g.C2 = b.C2; g.Zin = b.Zin;
  g.bias = b.bias; g.bias_dtype = D.dtype;
  g.a_rows = b.a_rows; g.a_rows_batch = b.a_rows_batch; g.a_rows_total = b.a_rows_total; g.a_rows_k = b.a_mn;   // the stored rows of A run along K when it is MN-major
  g.status = status_word;
  EC_CUDA(launch_gemm_simt(g, st));
  return EC_OK;
}

ec_status route_impl(const Dims& D, const void* X, const void* Wg, float* S, int32_t* I, float* G,
                     int32_t* row_ptr, int32_t* slots, char* ws, const WsLayout& W, cudaStream_t st,
                     int32_t* load = nullptr, int32_t* requested = nullptr) {
  bool done = false;
  if (D.dtype == EC_BF16) {
    TcGemmArgs t; memset(&t, 0, sizeof(t));
    t.A = X; t.B = Wg; t.a_mn_major = 0; t.b_mn_major = 1;
    t.M = (int)D.n; t.N = D.E; t.K = D.d; t.batches = 1; t.lda = D.d; t.ldb = D.E;
    t.epi = EPI_SOFTMAX; t.S = S; t.ldc = D.E; t.status = (int*)(ws + W.status);
    if (tc_gemm_supported(t)) { EC_CUDA(launch_gemm_tc(t, st)); done = true; }
  }
  if (!done) EC_CUDA(launch_gate_softmax_simt(D.dtype, X, Wg, S, D.n, D.d, D.E, st));
  prof_mark("gate_softmax", st);
  if (D.router == EC_ROUTER_TOKEN_TOP2) {            // Section 3.1's token choice as a contrast: tokens pick, experts have buffers
    int32_t* choice = (int32_t*)(ws + W.choice);
    EC_CUDA(launch_token_top2(S, D.n, D.E, choice, st));
    EC_CUDA(launch_token_admit(S, choice, D.ng, D.E, D.kg, D.groups, I, G, load, requested, st));
    prof_mark("token_choice", st);
    EC_CUDA(launch_inverse_index(I, D.n, D.slots, row_ptr, slots, ws + W.inverse, (int*)(ws + W.status), st));
    prof_mark("inverse_index", st);
    return EC_OK;
  }
  const float* keys = S;
  if (D.cap_b) {                                    // Section 3.3: TopK(A, k) instead of TopK(S^T, k)
    float* A = (float*)(ws + W.cap_A);
    EC_CUDA(launch_capped_assignment(S, D.ng, D.E, D.kg, D.groups, D.cap_b, D.cap_iters, (float)D.cap_lambda, A,
                                     ws + W.capped, st));
    prof_mark("capped_assignment", st);
    keys = A;
  }
  EC_CUDA(launch_topk(keys, D.ng, D.E, D.kg, D.groups, I, G, ws + W.topk, st));
  if (D.cap_b) EC_CUDA(launch_gather_gate(S, I, G, D.slots, D.k, D.E, D.n, (int*)(ws + W.status), st));      // the gate weights stay S at I
  prof_mark("topk", st);
  EC_CUDA(launch_inverse_index(I, D.n, D.slots, row_ptr, slots, ws + W.inverse, (int*)(ws + W.status), st));
  prof_mark("inverse_index", st);
  return EC_OK;
}

// Scratch of ec_route_static: lives in the library's own device image, so every GPU that loads
// the library holds these bytes until the process exits.  The name below is only a handle on the
// host; the device address is looked up once per device (static_scratch) and handed to the kernels.
static __device__ __align__(256) unsigned char g_route_scratch[EC_ROUTE_STATIC_SCRATCH_BYTES];

constexpr int kMaxDevices = 64;
std::mutex g_static_mu;
void* g_static_ptr[kMaxDevices] = {};

// Device address of g_route_scratch on the current device; resolved on the first call per device.
ec_status static_scratch(void** out) {
  int dev = -1;
  if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= kMaxDevices) return EC_ERR_CUDA;
  std::lock_guard<std::mutex> lock(g_static_mu);
  if (!g_static_ptr[dev]) {
    void* p = nullptr;
    if (cudaGetSymbolAddress(&p, g_route_scratch) != cudaSuccess || !p) return EC_ERR_CUDA;
    g_static_ptr[dev] = p;
  }
  *out = g_static_ptr[dev];
  return EC_OK;
}

// Bytes of scratch the routing stages alone use (the status word, the selection state and the
// inverse-index cursor); the backward buffers that share the workspace are not part of it.
size_t route_scratch_bytes(const Dims& D, const WsLayout& W) { (void)D; return W.fwd_end; }

}  // namespace

namespace ecmoe { void count_launch(int n) { g_launches += n; } }

extern "C" {

int64_t ec_capacity(const ec_config* c) {
  if (!c || c->E < 1 || c->n < 1 || !(c->c > 0.0)) return -1;
  const double kd = floor((double)c->n * c->c / (double)c->E + 1e-9);
  if (kd < 1.0 || kd > (double)c->n) return -1;
  return (int64_t)kd;
}

size_t ec_workspace_bytes(const ec_config* c) {
  Dims D; if (check_cfg(c, &D) != EC_OK) return 0;
  return ws_layout(D).total;
}

size_t ec_forward_only_workspace_bytes(const ec_config* c) {
  Dims D; if (check_cfg(c, &D) != EC_OK) return 0;
  return ws_layout(D).fwd_end + saved_layout(D, false).total;
}

size_t ec_saved_bytes(const ec_config* c) {
  Dims D; if (check_cfg(c, &D) != EC_OK) return 0;
  return saved_layout(D).total;
}

ec_status ec_saved_view(const ec_config* c, void* saved, ec_saved_ptrs* out) {
  Dims D; ec_status s = check_cfg(c, &D); if (s != EC_OK) return s;
  if (!saved || !out) return EC_ERR_INVALID_ARG;
  const SavedLayout L = saved_layout(D); char* b = (char*)saved;
  out->S = (float*)(b + L.S); out->I = (int32_t*)(b + L.I); out->G = (float*)(b + L.G);
  out->row_ptr = (int32_t*)(b + L.row_ptr); out->slots = (int32_t*)(b + L.slots);
  out->X_in = D.fuse ? nullptr : b + L.X_in; out->Z = b + L.Z; out->H = b + L.H; out->X_e = (float*)(b + L.X_e);
  out->load = D.router ? (int32_t*)(b + L.load) : nullptr;
  out->requested = D.router ? (int32_t*)(b + L.requested) : nullptr;
  return EC_OK;
}

ec_status ec_route(const ec_config* c, const void* X, const void* Wg, float* S, int32_t* I, float* G,
                   int32_t* row_ptr, int32_t* slots, void* ws, size_t ws_bytes, void* stream) {
  Dims D; ec_status s = check_cfg(c, &D); if (s != EC_OK) return s;
  if (D.router != EC_ROUTER_EXPERT_CHOICE) return EC_ERR_INVALID_ARG;      // ec_route_token_choice has the outputs for that
  if (!X || !Wg || !S || !I || !G || !row_ptr || !slots || !ws) return EC_ERR_INVALID_ARG;
  if (misaligned(X, 16) || misaligned(Wg, 16) || misaligned(S, 16) || misaligned(I, 16) || misaligned(G, 16) ||
      misaligned(row_ptr, 16) || misaligned(slots, 16) || misaligned(ws, kAlign)) return EC_ERR_INVALID_ARG;
  const WsLayout W = ws_layout(D);
  if (ws_bytes < W.total) return EC_ERR_WORKSPACE;
  cudaStream_t st = (cudaStream_t)stream;
  EC_CUDA(cudaMemsetAsync(ws, 0, sizeof(StatusWord), st));
  prof_begin(st, 0);
  return route_impl(D, X, Wg, S, I, G, row_ptr, slots, (char*)ws, W, st);
}

ec_status ec_route_token_choice(const ec_config* c, const void* X, const void* Wg, float* S, int32_t* I, float* G,
                                int32_t* row_ptr, int32_t* slots, int32_t* load, int32_t* requested, void* ws,
                                size_t ws_bytes, void* stream) {
  Dims D; ec_status s = check_cfg(c, &D); if (s != EC_OK) return s;
  if (D.router != EC_ROUTER_TOKEN_TOP2) return EC_ERR_INVALID_ARG;
  if (!X || !Wg || !S || !I || !G || !row_ptr || !slots || !load || !requested || !ws) return EC_ERR_INVALID_ARG;
  if (misaligned(X, 16) || misaligned(Wg, 16) || misaligned(S, 16) || misaligned(I, 16) || misaligned(G, 16) ||
      misaligned(row_ptr, 16) || misaligned(slots, 16) || misaligned(load, 4) || misaligned(requested, 4) ||
      misaligned(ws, kAlign)) return EC_ERR_INVALID_ARG;
  const WsLayout W = ws_layout(D);
  if (ws_bytes < W.total) return EC_ERR_WORKSPACE;
  cudaStream_t st = (cudaStream_t)stream;
  EC_CUDA(cudaMemsetAsync(ws, 0, sizeof(StatusWord), st));
  prof_begin(st, 0);
  return route_impl(D, X, Wg, S, I, G, row_ptr, slots, (char*)ws, W, st, load, requested);
}

ec_status ec_capped_assignment(const ec_config* c, const float* S, float* A, void* ws, size_t ws_bytes, void* stream) {
  Dims D; ec_status s = check_cfg(c, &D); if (s != EC_OK) return s;
  if (!D.cap_b) return EC_ERR_INVALID_ARG;
  if (!S || !A || !ws || misaligned(S, 16) || misaligned(A, 16) || misaligned(ws, kAlign)) return EC_ERR_INVALID_ARG;
  const WsLayout W = ws_layout(D);
  if (ws_bytes < W.total) return EC_ERR_WORKSPACE;
  cudaStream_t st = (cudaStream_t)stream;
  EC_CUDA(cudaMemsetAsync(ws, 0, sizeof(StatusWord), st));
  prof_begin(st, 0);
  EC_CUDA(launch_capped_assignment(S, D.ng, D.E, D.kg, D.groups, D.cap_b, D.cap_iters, (float)D.cap_lambda, A,
                                   (char*)ws + W.capped, st));
  prof_mark("capped_assignment", st);
  return EC_OK;
}

ec_status ec_shuffle(const ec_config* c, const void* X, const int32_t* I, void* X_in, void* stream) {
  Dims D; ec_status s = check_cfg(c, &D); if (s != EC_OK) return s;
  if (!X || !I || !X_in) return EC_ERR_INVALID_ARG;
  if (misaligned(X, 16) || misaligned(I, 16) || misaligned(X_in, 16)) return EC_ERR_INVALID_ARG;
  cudaStream_t st = (cudaStream_t)stream;
  prof_begin(st, 0);
  EC_CUDA(launch_gather(D.dtype, X, I, X_in, D.slots, D.d, D.n, nullptr, st));
  prof_mark("gather", st);
  return EC_OK;
}

ec_status ec_unshuffle(const ec_config* c, const float* X_e, const float* G, const int32_t* row_ptr,
                       const int32_t* slots, void* X_out, void* stream) {
  Dims D; ec_status s = check_cfg(c, &D); if (s != EC_OK) return s;
  if (!X_e || !G || !row_ptr || !slots || !X_out) return EC_ERR_INVALID_ARG;
  if (misaligned(X_e, 16) || misaligned(G, 16) || misaligned(row_ptr, 16) || misaligned(slots, 16) ||
      misaligned(X_out, 16)) return EC_ERR_INVALID_ARG;
  cudaStream_t st = (cudaStream_t)stream;
  prof_begin(st, 0);
  EC_CUDA(launch_combine(D.dtype, X_e, G, row_ptr, slots, X_out, D.n, D.d, D.slots, nullptr, st));
  prof_mark("combine", st);
  return EC_OK;
}

size_t ec_route_static_bytes(const ec_config* c) {
  Dims D; if (check_cfg(c, &D) != EC_OK) return 0;
  return route_scratch_bytes(D, ws_layout(D));
}

ec_status ec_route_static(const ec_config* c, const void* X, const void* Wg, float* S, int32_t* I, float* G,
                          int32_t* row_ptr, int32_t* slots, void* stream) {
  Dims D; ec_status s = check_cfg(c, &D); if (s != EC_OK) return s;
  if (D.router != EC_ROUTER_EXPERT_CHOICE) return EC_ERR_INVALID_ARG;
  if (!X || !Wg || !S || !I || !G || !row_ptr || !slots) return EC_ERR_INVALID_ARG;
  if (misaligned(X, 16) || misaligned(Wg, 16) || misaligned(S, 16) || misaligned(I, 16) || misaligned(G, 16) ||
      misaligned(row_ptr, 16) || misaligned(slots, 16)) return EC_ERR_INVALID_ARG;
  const WsLayout W = ws_layout(D);
  if (route_scratch_bytes(D, W) > (size_t)EC_ROUTE_STATIC_SCRATCH_BYTES) return EC_ERR_WORKSPACE;
  void* ws = nullptr;
  if ((s = static_scratch(&ws)) != EC_OK) return s;
  cudaStream_t st = (cudaStream_t)stream;
  // The array keeps whatever the previous call left: the status word is cleared here, and the
  // routing stages clear their own counters, histograms and cursors before they use them.
  EC_CUDA(cudaMemsetAsync(ws, 0, sizeof(StatusWord), st));
  prof_begin(st, 0);
  return route_impl(D, X, Wg, S, I, G, row_ptr, slots, (char*)ws, W, st);
}

ec_status ec_moe_forward(const ec_config* c, const void* X, const void* Wg, const void* W1, const void* W2,
                         const void* b1, const void* b2, void* X_out, void* saved, size_t saved_bytes, void* ws,
                         size_t ws_bytes, void* stream) {
  Dims D; ec_status s = check_cfg(c, &D); if (s != EC_OK) return s;
  if (!X || !Wg || !W1 || !W2 || !X_out || !ws) return EC_ERR_INVALID_ARG;
  const bool keep = saved != nullptr;                // else forward only: nothing is kept for a backward pass
  if (!keep && saved_bytes != 0) return EC_ERR_INVALID_ARG;
  if (misaligned(X, 16) || misaligned(Wg, 16) || misaligned(W1, 16) || misaligned(W2, 16) || misaligned(X_out, 16) ||
      misaligned(b1, 16) || misaligned(b2, 16) || misaligned(saved, kAlign) || misaligned(ws, kAlign)) return EC_ERR_INVALID_ARG;
  const WsLayout W = ws_layout(D); const SavedLayout L = saved_layout(D, keep);
  if (keep ? (ws_bytes < W.total || saved_bytes < L.total) : ws_bytes < W.fwd_end + L.total) return EC_ERR_WORKSPACE;
  cudaStream_t st = (cudaStream_t)stream;
  char* w = (char*)ws; char* sv = keep ? (char*)saved : w + W.fwd_end;    // forward only: the intermediates follow the routing scratch
  float* S = (float*)(sv + L.S); int32_t* I = (int32_t*)(sv + L.I); float* G = (float*)(sv + L.G);
  int32_t* row_ptr = (int32_t*)(sv + L.row_ptr); int32_t* slots = (int32_t*)(sv + L.slots);
  void* X_in = sv + L.X_in; void* Z = keep ? sv + L.Z : nullptr; void* H = sv + L.H; float* X_e = (float*)(sv + L.X_e);
  int* status = (int*)(w + W.status);
  EC_CUDA(cudaMemsetAsync(ws, 0, sizeof(StatusWord), st));
  prof_begin(st, 0);
  // token-choice contrast: slots filled per expert; with one routing group they are a prefix of the expert's buffer and
  // the tensor-core GEMMs skip what lies beyond
  int32_t* load = D.router ? (int32_t*)(sv + L.load) : nullptr;
  int32_t* requested = D.router ? (int32_t*)(sv + L.requested) : nullptr;
  const int32_t* rag = D.router && D.groups == 1 ? load : nullptr;
  if ((s = route_impl(D, X, Wg, S, I, G, row_ptr, slots, w, W, st, load, requested)) != EC_OK) return s;
  if (!D.fuse) {
    EC_CUDA(launch_gather(D.dtype, X, I, X_in, D.slots, D.d, D.n, status, st));
    prof_mark("gather", st);
  }
  const int64_t kd = D.k * D.d, kf = D.k * D.dff, df = (int64_t)D.d * D.dff;
  // Z = X_in[i] . W1[i],  H = GeLU(Z); with fuse_gather X_in[i] is rows I[i, :] of X read in place
  BatchedGemm g1 = {X_in, 0, D.d, kd, W1, 1, D.dff, df, Z, D.dff, kf, (int)D.k, D.dff, D.d, D.E, EPI_GELU, H, nullptr, 0, rag, 1, b1};
  if (D.fuse) { g1.A = X; g1.batch_a = 0; g1.a_rows = I; g1.a_rows_batch = D.k; g1.a_rows_total = D.n; }
  if ((s = run_gemm(D, g1, status, st)) != EC_OK) return s;
  prof_mark("gemm1_gelu", st);
  // X_e = H[i] . W2[i]^T, kept in fp32
  BatchedGemm g2 = {H, 0, D.dff, kf, W2, 0, D.dff, df, X_e, D.d, kd, (int)D.k, D.d, D.dff, D.E, EPI_STORE, nullptr, nullptr, 1, rag, 1, b2};
  if ((s = run_gemm(D, g2, status, st)) != EC_OK) return s;
  prof_mark("gemm2", st);
  EC_CUDA(launch_combine(D.dtype, X_e, G, row_ptr, slots, X_out, D.n, D.d, D.slots, status, st));
  prof_mark("combine", st);
  return EC_OK;
}

ec_status ec_moe_backward(const ec_config* c, const void* X, const void* Wg, const void* W1, const void* W2,
                          const void* dX_out, const void* saved, size_t saved_bytes, void* dX, void* dWg,
                          void* dW1, void* dW2, void* db1, void* db2, void* ws, size_t ws_bytes, void* stream) {
  Dims D; ec_status s = check_cfg(c, &D); if (s != EC_OK) return s;
  if (!X || !Wg || !W1 || !W2 || !dX_out || !saved || !dX || !dWg || !dW1 || !dW2 || !ws) return EC_ERR_INVALID_ARG;
  if (misaligned(X, 16) || misaligned(Wg, 16) || misaligned(W1, 16) || misaligned(W2, 16) || misaligned(dX_out, 16) ||
      misaligned(dX, 16) || misaligned(dWg, 16) || misaligned(dW1, 16) || misaligned(dW2, 16) ||
      misaligned(db1, 16) || misaligned(db2, 16) || misaligned(saved, kAlign) || misaligned(ws, kAlign)) return EC_ERR_INVALID_ARG;
  const WsLayout W = ws_layout(D); const SavedLayout L = saved_layout(D);
  if (ws_bytes < W.total || saved_bytes < L.total) return EC_ERR_WORKSPACE;
  cudaStream_t st = (cudaStream_t)stream;
  const char* sv = (const char*)saved; char* w = (char*)ws;
  const float* S = (const float*)(sv + L.S); const int32_t* I = (const int32_t*)(sv + L.I);
  const float* G = (const float*)(sv + L.G);
  const int32_t* row_ptr = (const int32_t*)(sv + L.row_ptr); const int32_t* slots = (const int32_t*)(sv + L.slots);
  const void* X_in = sv + L.X_in; const void* Z = sv + L.Z; const void* H = sv + L.H; const float* X_e = (const float*)(sv + L.X_e);
  void* dX_e = w + W.dX_e; float* dG = (float*)(w + W.dG); void* dZ = w + W.dZ; void* dX_in = w + W.dX_in;
  void* dL = w + W.dL; float* part = (float*)(w + W.dWg_part);
  int* status = (int*)(w + W.status);
  const int32_t* rag = D.router && D.groups == 1 ? (const int32_t*)(sv + L.load) : nullptr;   // see ec_moe_forward
  EC_CUDA(cudaMemsetAsync(ws, 0, sizeof(StatusWord), st));
  const int64_t kd = D.k * D.d, kf = D.k * D.dff, df = (int64_t)D.d * D.dff;
  // Eq. 4 backward: dX_e, dG
  prof_begin(st, 1);
  EC_CUDA(launch_bwd_combine(D.dtype, dX_out, X_e, G, I, dX_e, dG, D.slots, D.d, D.n, status, st));
  prof_mark("bwd_combine", st);
  // dZ = (dX_e[i] . W2[i]) * GeLU'(Z)
  BatchedGemm g3 = {dX_e, 0, D.d, kd, W2, 1, D.dff, df, dZ, D.dff, kf, (int)D.k, D.dff, D.d, D.E, EPI_GELU_GRAD, nullptr, Z, 0, rag, 1, nullptr};
  if ((s = run_gemm(D, g3, status, st)) != EC_OK) return s;
  prof_mark("gemm_dZ", st);
  if (db1 || db2) {                                  // gradients of the bias terms: sums over an expert's slots of dZ and of dX_e
    if (db1) EC_CUDA(launch_column_sums(D.dtype, dZ, db1, D.E, D.k, D.dff, rag, st));
    if (db2) EC_CUDA(launch_column_sums(D.dtype, dX_e, db2, D.E, D.k, D.d, rag, st));
    prof_mark("bias_grads", st);
  }
  // dW2[i] = dX_e[i]^T . H[i]
  BatchedGemm g4 = {dX_e, 1, D.d, kd, H, 1, D.dff, kf, dW2, D.dff, df, D.d, D.dff, (int)D.k, D.E, EPI_STORE, nullptr, nullptr, 0, rag, 2, nullptr};
  if ((s = run_gemm(D, g4, status, st)) != EC_OK) return s;
  prof_mark("gemm_dW2", st);
  // dW1[i] = X_in[i]^T . dZ[i]
  BatchedGemm g5 = {X_in, 1, D.d, kd, dZ, 1, D.dff, kf, dW1, D.dff, df, D.d, D.dff, (int)D.k, D.E, EPI_STORE, nullptr, nullptr, 0, rag, 2, nullptr};
  if (D.fuse) { g5.A = X; g5.batch_a = 0; g5.a_rows = I; g5.a_rows_batch = D.k; g5.a_rows_total = D.n; }   // X_in[i] again read from X through I
  if ((s = run_gemm(D, g5, status, st)) != EC_OK) return s;
  prof_mark("gemm_dW1", st);
  // dX_in[i] = dZ[i] . W1[i]^T
  BatchedGemm g6 = {dZ, 0, D.dff, kf, W1, 0, D.dff, df, dX_in, D.d, kd, (int)D.k, D.d, D.dff, D.E, EPI_STORE, nullptr, nullptr, 0, rag, 1, nullptr};
  if ((s = run_gemm(D, g6, status, st)) != EC_OK) return s;
  prof_mark("gemm_dXin", st);
  // softmax backward: dL [n, E]; bf16 when the two gate-gradient products below run on tensor cores
  const int P = dwg_splits(D);
  TcGemmArgs tw; memset(&tw, 0, sizeof(tw));          // dWg = X^T . dL, cut along the tokens
  const int64_t cut = (((D.n + P - 1) / P) + 63) / 64 * 64;
  tw.A = X; tw.a_mn_major = 1; tw.lda = D.d; tw.B = dL; tw.b_mn_major = 1; tw.ldb = D.E;
  tw.M = D.d; tw.N = D.E; tw.K = (int)cut; tw.batches = P; tw.k_split = 1; tw.k_total = D.n;
  tw.epi = EPI_STORE; tw.c_f32 = 1; tw.C = part; tw.ldc = D.E; tw.batch_c = (int64_t)D.d * D.E; tw.status = status;
  TcGemmArgs tx; memset(&tx, 0, sizeof(tx));          // dX = dL . Wg^T + rows of dX_in
  tx.A = dL; tx.a_mn_major = 0; tx.lda = D.E; tx.B = Wg; tx.b_mn_major = 0; tx.ldb = D.E;
  tx.M = (int)D.n; tx.N = D.d; tx.K = D.E; tx.batches = 1;
  tx.epi = EPI_ADD_SLOTS; tx.C = dX; tx.ldc = D.d; tx.status = status;
  tx.row_ptr = row_ptr; tx.slots = slots; tx.rows = dX_in; tx.ld_rows = D.d; tx.slots_total = D.slots;
  const bool tc_gate = D.dtype == EC_BF16 && tc_gemm_supported(tw) && tc_gemm_supported(tx);     // mirrored by gate_grads_on_tc()
  EC_CUDA(launch_bwd_softmax(S, dG, row_ptr, slots, dL, tc_gate ? 1 : 0, D.n, D.E, D.k, status, st));
  prof_mark("bwd_softmax", st);
  if (tc_gate) {
    EC_CUDA(launch_gemm_tc(tw, st));
    EC_CUDA(launch_reduce_partials(D.dtype, part, dWg, P, (int64_t)D.d * D.E, st));
    prof_mark("dWg", st);
    EC_CUDA(launch_gemm_tc(tx, st));
    prof_mark("dX", st);
    return EC_OK;
  }
  // dWg = X^T . dL, split over the tokens into fixed chunks and summed in a fixed order
  {
    const int64_t chunk = (D.n + P - 1) / P;
    GemmArgs g; memset(&g, 0, sizeof(g));
    g.A = X; g.B = dL; g.C = part; g.a_dtype = D.dtype; g.b_dtype = EC_F32; g.c_dtype = EC_F32;
    g.M = D.d; g.N = D.E; g.K = (int)chunk; g.batches = P; g.k_limit = D.n;
    g.sam = 1; g.sak = D.d; g.sbk = D.E; g.sbn = 1; g.ldc = D.E;
    g.batch_a = chunk * D.d; g.batch_b = chunk * D.E; g.batch_c = (int64_t)D.d * D.E;
    g.epi = EPI_STORE;
    EC_CUDA(launch_gemm_simt(g, st));
    EC_CUDA(launch_reduce_partials(D.dtype, part, dWg, P, (int64_t)D.d * D.E, st));
    prof_mark("dWg", st);
  }
  // dX = dL . Wg^T + sum over the slots of each token of dX_in
  {
    GemmArgs g; memset(&g, 0, sizeof(g));
    g.A = dL; g.B = Wg; g.C = dX; g.a_dtype = EC_F32; g.b_dtype = D.dtype; g.c_dtype = D.dtype;
    g.M = (int)D.n; g.N = D.d; g.K = D.E; g.batches = 1;
    g.sam = D.E; g.sak = 1; g.sbk = 1; g.sbn = D.E; g.ldc = D.d;
    g.epi = EPI_ADD_SLOTS; g.row_ptr = row_ptr; g.slots = slots; g.rows = dX_in; g.ld_rows = D.d;
    g.slots_total = D.slots; g.status = status;
    EC_CUDA(launch_gemm_simt(g, st));
    prof_mark("dX", st);
  }
  return EC_OK;
}

ec_status ec_expert_gemm(const ec_config* c, int kind, const void* A, const void* B, void* C, void* ws, size_t ws_bytes,
                         void* stream) {
  Dims D; ec_status s = check_cfg(c, &D); if (s != EC_OK) return s;
  if (kind != EC_GEMM_XW1 && kind != EC_GEMM_HW2T && kind != EC_GEMM_ATB) return EC_ERR_INVALID_ARG;
  if (!A || !B || !C || !ws || misaligned(A, 16) || misaligned(B, 16) || misaligned(C, 16) || misaligned(ws, kAlign))
    return EC_ERR_INVALID_ARG;
  if (ws_bytes < ws_layout(D).total) return EC_ERR_WORKSPACE;
  cudaStream_t st = (cudaStream_t)stream;
  EC_CUDA(cudaMemsetAsync(ws, 0, sizeof(StatusWord), st));
  const int64_t kd = D.k * D.d, kf = D.k * D.dff, df = (int64_t)D.d * D.dff;
  BatchedGemm g;
  if (kind == EC_GEMM_XW1) g = {A, 0, D.d, kd, B, 1, D.dff, df, C, D.dff, kf, (int)D.k, D.dff, D.d, D.E, EPI_STORE, nullptr, nullptr, 0, nullptr, 0, nullptr};
  else if (kind == EC_GEMM_HW2T) g = {A, 0, D.dff, kf, B, 0, D.dff, df, C, D.d, kd, (int)D.k, D.d, D.dff, D.E, EPI_STORE, nullptr, nullptr, 0, nullptr, 0, nullptr};
  else g = {A, 1, D.d, kd, B, 1, D.dff, kf, C, D.dff, df, D.d, D.dff, (int)D.k, D.E, EPI_STORE, nullptr, nullptr, 0, nullptr, 0, nullptr};
  prof_begin(st, 0);
  s = run_gemm(D, g, (int*)ws, st);
  prof_mark("expert_gemm", st);
  return s;
}

ec_status ec_validate_routing(const ec_config* c, const int32_t* I, const int32_t* row_ptr, const int32_t* slots,
                              int64_t* violations, void* ws, size_t ws_bytes, void* stream) {
  Dims D; ec_status s = check_cfg(c, &D); if (s != EC_OK) return s;
  if (!I || !row_ptr || !slots || !violations || !ws || misaligned(ws, kAlign)) return EC_ERR_INVALID_ARG;
  if (ws_bytes < ws_layout(D).total) return EC_ERR_WORKSPACE;
  cudaStream_t st = (cudaStream_t)stream;
  int* counters = (int*)ws + 8;                        // inside the status block, past the words the kernels use
  EC_CUDA(launch_validate_routing(I, row_ptr, slots, D.n, D.ng, D.E, D.k, D.kg, D.groups, D.router == EC_ROUTER_TOKEN_TOP2 ? 1 : 0,
                                  counters, st));
  int h[2] = {0, 0};
  EC_CUDA(cudaMemcpyAsync(h, counters, sizeof(h), cudaMemcpyDeviceToHost, st));
  EC_CUDA(cudaStreamSynchronize(st));
  *violations = h[0];
  return EC_OK;
}

namespace {
// Whether ec_moe_backward runs dWg and dX on the tensor cores (dL is then bf16): the shape part of its decision, the
// pointers being 256-byte aligned parts of the workspace and 16-byte aligned arguments.
bool gate_grads_on_tc(const Dims& D) {
  if (D.dtype != EC_BF16) return false;
  const int P = dwg_splits(D);
  const int64_t cut = (((D.n + P - 1) / P) + 63) / 64 * 64;
  TcGemmArgs tw; memset(&tw, 0, sizeof(tw));
  tw.A = tw.B = tw.C = (void*)256; tw.a_mn_major = 1; tw.lda = D.d; tw.b_mn_major = 1; tw.ldb = D.E;
  tw.M = D.d; tw.N = D.E; tw.K = (int)cut; tw.batches = P; tw.k_split = 1; tw.k_total = D.n;
  tw.epi = EPI_STORE; tw.c_f32 = 1; tw.ldc = D.E; tw.batch_c = (int64_t)D.d * D.E;
  TcGemmArgs tx; memset(&tx, 0, sizeof(tx));
  tx.A = tx.B = tx.C = (void*)256; tx.lda = D.E; tx.ldb = D.E; tx.M = (int)D.n; tx.N = D.d; tx.K = D.E; tx.batches = 1;
  tx.epi = EPI_ADD_SLOTS; tx.ldc = D.d; tx.row_ptr = (const int32_t*)256; tx.slots = (const int32_t*)256; tx.rows = (void*)256; tx.ld_rows = D.d;
  return tc_gemm_supported(tw) && tc_gemm_supported(tx);
}
}  // namespace

ec_status ec_backward_view(const ec_config* c, void* ws, ec_backward_ptrs* out) {
  Dims D; ec_status s = check_cfg(c, &D); if (s != EC_OK) return s;
  if (!ws || !out) return EC_ERR_INVALID_ARG;
  const WsLayout W = ws_layout(D); char* w = (char*)ws;
  out->dX_e = w + W.dX_e; out->dG = (float*)(w + W.dG); out->dZ = w + W.dZ; out->dX_in = w + W.dX_in; out->dL = w + W.dL;
  out->dL_is_bf16 = gate_grads_on_tc(D) ? 1 : 0;
  return EC_OK;
}

int ec_debug_build(void) {
#ifdef EC_DEBUG
  return 1;
#else
  return 0;
#endif
}

ec_status ec_read_status(const void* ws, void* stream) {
  if (!ws) return EC_ERR_INVALID_ARG;
  StatusWord h;
  if (cudaStreamSynchronize((cudaStream_t)stream) != cudaSuccess) return EC_ERR_CUDA;
  if (cudaMemcpy(&h, ws, sizeof(h), cudaMemcpyDeviceToHost) != cudaSuccess) return EC_ERR_CUDA;
  return h.code == 0 ? EC_OK : (h.code == EC_ERR_TIMEOUT ? EC_ERR_TIMEOUT : (h.code == EC_ERR_INDEX ? EC_ERR_INDEX : EC_ERR_CUDA));
}

const char* ec_status_string(ec_status s) {
  switch (s) {
    case EC_OK: return "ok";
    case EC_ERR_INVALID_ARG: return "invalid argument";
    case EC_ERR_UNSUPPORTED: return "unsupported configuration";
    case EC_ERR_WORKSPACE: return "workspace or saved buffer too small";
    case EC_ERR_CUDA: return "CUDA call failed";
    case EC_ERR_TIMEOUT: return "a bounded device-side wait expired";
    case EC_ERR_INDEX: return "an index read from I, row_ptr or slots was out of range";
  }
  return "unknown status";
}

long long ec_launch_count(void) { return g_launches.load(); }

void ec_profile_enable(int on) { g_prof_enabled = on != 0; g_prof[0].count = g_prof[1].count = 0; }

int ec_profile_read(float* ms, const char** names, int max_stages) {
  if (!g_prof_enabled) return 0;
  int nst = 0;
  for (int kind = 0; kind < 2; ++kind) {
    Profile& P = g_prof[kind];
    if (P.count == 0) continue;
    if (cudaEventSynchronize(P.ev[P.count]) != cudaSuccess) return -1;
    for (int i = 0; i < P.count && nst < max_stages; ++i, ++nst) {
      float t = 0.f;
      if (cudaEventElapsedTime(&t, P.ev[i], P.ev[i + 1]) != cudaSuccess) return -1;
      if (ms) ms[nst] = t;
      if (names) names[nst] = P.names[i];
    }
    P.count = 0;
  }
  return nst;
}

int ec_uses_tensor_cores(const ec_config* c) {
  Dims D; if (check_cfg(c, &D) != EC_OK || D.dtype != EC_BF16) return 0;
  TcGemmArgs t; memset(&t, 0, sizeof(t));
  t.a_mn_major = 0; t.b_mn_major = 1; t.M = (int)D.k; t.N = D.dff; t.K = D.d; t.batches = D.E;
  t.lda = D.d; t.ldb = D.dff; t.ldc = D.dff; t.epi = EPI_GELU;
  t.A = t.B = t.C = (void*)16;   // shape query only
  return tc_gemm_supported(t) ? 1 : 0;
}

}  // extern "C"
