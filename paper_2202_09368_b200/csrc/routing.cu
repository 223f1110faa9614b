// Routing, shuffle and unshuffle kernels of the expert-choice layer (Section 3.2, Eq. 2-4)
// and the element-wise parts of its backward pass.  Everything here is bandwidth- or
// latency-bound integer / fp32 work; the dense contractions live in gemm_*.cu.
#include "internal.h"

#include <string.h>

namespace ecmoe {

// ------------------------------------------------------------------------------------------
// small helpers
// ------------------------------------------------------------------------------------------
__device__ __forceinline__ float ld_f(const float* p, int64_t i) { return p[i]; }
__device__ __forceinline__ float ld_f(const bf16* p, int64_t i) { return __bfloat162float(p[i]); }

template <typename T> struct Vec;            // one 16-byte vector of T
template <> struct Vec<float> {
  static constexpr int N = 4;
  __device__ static void unpack(const uint4& v, float* f) {
    f[0] = __uint_as_float(v.x); f[1] = __uint_as_float(v.y);
    f[2] = __uint_as_float(v.z); f[3] = __uint_as_float(v.w);
  }
  __device__ static uint4 pack(const float* f) {
    return make_uint4(__float_as_uint(f[0]), __float_as_uint(f[1]), __float_as_uint(f[2]),
                      __float_as_uint(f[3]));
  }
};
template <> struct Vec<bf16> {
  static constexpr int N = 8;
  __device__ static void unpack(const uint4& v, float* f) {
    const unsigned w[4] = {v.x, v.y, v.z, v.w};
#pragma unroll
    for (int i = 0; i < 4; ++i) {            // bf16 -> fp32 is a 16-bit shift
      f[2 * i] = __uint_as_float(w[i] << 16);
      f[2 * i + 1] = __uint_as_float(w[i] & 0xFFFF0000u);
    }
  }
  __device__ static uint4 pack(const float* f) {
    unsigned w[4];
#pragma unroll
    for (int i = 0; i < 4; ++i) {
      __nv_bfloat162 p = __floats2bfloat162_rn(f[2 * i], f[2 * i + 1]);
      w[i] = *reinterpret_cast<unsigned*>(&p);
    }
    return make_uint4(w[0], w[1], w[2], w[3]);
  }
};

static inline unsigned grid_for(int64_t work, int threads, int64_t cap = 148 * 16) {
  int64_t b = (work + threads - 1) / threads;
  if (b < 1) b = 1;
  if (b > cap) b = cap;
  return (unsigned)b;
}

// ------------------------------------------------------------------------------------------
// Gate, Eq. 2: S = Softmax(X . Wg) over the experts of each token.  FMA version (fp32 path and
// shapes the tensor-core kernel does not take).  One CTA handles TT tokens; the logits of the
// TT x E (token, expert) pairs are spread over the threads.
// ------------------------------------------------------------------------------------------
constexpr int kGateTT = 8, kGateDC = 512, kGateThreads = 256, kGateMaxE = 256;

template <typename T>
__global__ void __launch_bounds__(kGateThreads)
gate_softmax_simt_kernel(const T* __restrict__ X, const T* __restrict__ Wg, float* __restrict__ S,
                         int64_t n, int d, int E) {
  __shared__ float Xs[kGateTT][kGateDC];
  __shared__ float Ls[kGateTT][kGateMaxE];
  const int64_t t0 = (int64_t)blockIdx.x * kGateTT;
  const int tid = threadIdx.x;
  constexpr int R = kGateTT * kGateMaxE / kGateThreads;
  float acc[R];
#pragma unroll
  for (int r = 0; r < R; ++r) acc[r] = 0.f;
  const int pairs = kGateTT * E;
  for (int d0 = 0; d0 < d; d0 += kGateDC) {
    const int dc = min(kGateDC, d - d0);
    for (int idx = tid; idx < kGateTT * dc; idx += kGateThreads) {
      const int tt = idx / dc, dd = idx % dc;
      const int64_t t = t0 + tt;
      Xs[tt][dd] = t < n ? ld_f(X, t * d + d0 + dd) : 0.f;
    }
    __syncthreads();
#pragma unroll
    for (int r = 0; r < R; ++r) {
      const int p = tid + r * kGateThreads;
      if (p < pairs) {
        const int tt = p / E, i = p % E;
        float a = acc[r];
        for (int dd = 0; dd < dc; ++dd) a = fmaf(Xs[tt][dd], ld_f(Wg, (int64_t)(d0 + dd) * E + i), a);
        acc[r] = a;
      }
    }
    __syncthreads();
  }
#pragma unroll
  for (int r = 0; r < R; ++r) {
    const int p = tid + r * kGateThreads;
    if (p < pairs) Ls[p / E][p % E] = acc[r];
  }
  __syncthreads();
  const int warp = tid >> 5, lane = tid & 31;     // one warp per token
  const int64_t t = t0 + warp;
  if (warp < kGateTT && t < n) {
    float mx = -INFINITY;
    for (int i = lane; i < E; i += 32) mx = fmaxf(mx, Ls[warp][i]);
    for (int o = 16; o; o >>= 1) mx = fmaxf(mx, __shfl_xor_sync(0xffffffffu, mx, o));
    float sum = 0.f;
    for (int i = lane; i < E; i += 32) { const float e = expf(Ls[warp][i] - mx); Ls[warp][i] = e; sum += e; }
    for (int o = 16; o; o >>= 1) sum += __shfl_xor_sync(0xffffffffu, sum, o);
    const float inv = 1.f / sum;
    for (int i = lane; i < E; i += 32) S[t * E + i] = Ls[warp][i] * inv;
  }
}

cudaError_t launch_gate_softmax_simt(int dtype, const void* X, const void* Wg, float* S, int64_t n,
                                     int d, int E, cudaStream_t st) {
  const unsigned grid = (unsigned)((n + kGateTT - 1) / kGateTT);
  count_launch();
  if (dtype == 0)
    gate_softmax_simt_kernel<float><<<grid, kGateThreads, 0, st>>>((const float*)X, (const float*)Wg, S, n, d, E);
  else
    gate_softmax_simt_kernel<bf16><<<grid, kGateThreads, 0, st>>>((const bf16*)X, (const bf16*)Wg, S, n, d, E);
  return cudaGetLastError();
}

// ------------------------------------------------------------------------------------------
// Column top-k, Eq. 2: G, I = TopK(S^T, k).
//
// Every (token t, expert i) entry gets the 64-bit key  (~bits(S[t,i]) << 32) | t.  0 <= S <= 1, so its
// bit pattern is below 2^30 and monotone in its value: a smaller key is a larger score, and among
// equal scores a lower token.  Keys of one expert are distinct, so "the k smallest keys, ascending"
// is the unique answer with ties broken toward the lower token and slots listed by descending score.
//
// Routing groups (several independent groups of n tokens) multiply the columns: every (group, expert) pair is
// selected on its own and lands in its expert's row of I and G at the group's offset.
//
// Groups of up to kSmallN tokens with k up to one sort tile take one launch (topk_small_kernel, further down:
// one CTA per column does everything in shared memory).  Larger ones take the path described next.
//
// Selection is a most-significant-digit radix select over the 30 significant score bits, 10 bits a
// pass, run for all experts at once: a pass histograms its digit of the keys that still match the
// expert's prefix (in shared memory, merged into one global histogram per expert), and the last
// CTA of a column chunk to finish picks the bucket in which the k-th key lies.  An expert leaves
// the passes as soon as that bucket is small: either it holds exactly the keys still wanted, or at
// most kCandCap keys, the candidates, from which the final sort picks the best.  With distinct
// scores that is after two passes over S.  Experts still undecided after the three score passes
// have more than kCandCap exactly equal scores at the threshold: there the lowest tokens win, and
// one CTA per such expert walks the column in token order and takes the first ones.  One more pass
// over S then copies the winners (and candidates) out, and a bitonic network sorts each expert's keys.
//
// scratch, with C = groups * E columns: [SelState C][hist C*1024 u32][counters passes*groups*chunks u32]
//          [cursors 2C u32] (zeroed per call) [candidates C*kCandCap u64][keys C*kpad u64]
// ------------------------------------------------------------------------------------------
constexpr int kHistThreads = 1024;
constexpr int kBins = 1 << kRadixBits;
constexpr int kHistSmemBytes = (kBins + kBins / 32) * kTopkChunk * 4;   // [bin][column of the chunk]; the selection step re-uses it padded
constexpr unsigned long long kKeyTop = 3ull << 62;              // the two always-set top bits of a key

__device__ __forceinline__ unsigned long long make_key(float s, int64_t t) {
  return ((unsigned long long)(~__float_as_uint(s)) << 32) | (unsigned long long)(unsigned)t;
}

struct TopkLayout {
  size_t off_state, off_hist, off_counters, off_cursor, off_cand, off_keys, zero_bytes, total;
  int chunks; int64_t kpad;
};
// E experts of each of `groups` routing groups: groups * E independent columns ("virtual experts", group-major)
static TopkLayout topk_layout(int64_t n, int E, int64_t k, int groups) {
  TopkLayout L;
  L.chunks = (E + kTopkChunk - 1) / kTopkChunk;
  const size_t VE = (size_t)groups * E;
  L.kpad = 1; while (L.kpad < k) L.kpad <<= 1;
  size_t o = 0;
  auto take = [&](size_t b) { size_t r = o; o += (b + 255) & ~(size_t)255; return r; };
  L.off_state = take(sizeof(SelState) * VE);
  L.off_hist = take(VE * kBins * 4);
  L.off_counters = take((size_t)kRadixPasses * groups * L.chunks * 4);
  L.off_cursor = take(2 * VE * 4);
  L.zero_bytes = o;                       // everything up to here starts at zero
  L.off_cand = take(VE * kCandCap * 8);
  L.off_keys = take(VE * L.kpad * 8);
  L.total = o;
  return L;
}
size_t topk_scratch_bytes(int64_t n, int E, int64_t k, int groups) { return topk_layout(n, E, k, groups).total; }

__device__ __forceinline__ int pow2_at_least(int v) { int p = 1; while (p < v) p <<= 1; return p; }

// Walks the [t0, t1) x [c0, c0 + cw) slab of S with every thread of the CTA.  A thread always sees the same
// columns (four consecutive ones with VEC, one without): slab_first_col() tells it which, or -1 for none,
// and f(score, token, j) gets the j-th of them, j a compile-time 0..3, so per-column state can sit in
// registers.  VEC: 16-byte loads (E a multiple of 4), else scalar.  Four independent loads per thread
// are in flight.
template <bool VEC>
__device__ __forceinline__ int slab_first_col(int cw) {
  const int lane = threadIdx.x & 31;
  if constexpr (VEC) { const int lpr = pow2_at_least((cw + 3) >> 2); const int g = (lane % lpr) * 4; return g < cw ? g : -1; }
  else { const int cwp = pow2_at_least(cw); const int cc = lane % cwp; return cc < cw ? cc : -1; }
}
template <bool VEC, typename F>
__device__ __forceinline__ void for_slab(const float* __restrict__ S, int E, int c0, int cw, int64_t t0, int64_t t1, F&& f) {
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31, nwarps = blockDim.x >> 5;
  constexpr int U = 4;
  if constexpr (VEC) {
    const int lpr = pow2_at_least((cw + 3) >> 2), rpw = 32 / lpr;      // lanes per row, rows per warp
    const int r = lane / lpr, g = (lane % lpr) * 4;
    if (g >= cw) return;
    const int64_t step = (int64_t)nwarps * rpw;
    for (int64_t t = t0 + warp * rpw + r; t < t1; t += step * U) {
      float4 v[U];
#pragma unroll
      for (int u = 0; u < U; ++u)
        if (t + u * step < t1) v[u] = *reinterpret_cast<const float4*>(S + (t + u * step) * E + c0 + g);
#pragma unroll
      for (int u = 0; u < U; ++u)
        if (t + u * step < t1) {
          const int64_t tt = t + u * step;
          f(v[u].x, tt, 0); f(v[u].y, tt, 1); f(v[u].z, tt, 2); f(v[u].w, tt, 3);
        }
    }
  } else {
    const int cwp = pow2_at_least(cw), rpw = 32 / cwp;
    const int r = lane / cwp, cc = lane % cwp;
    if (cc >= cw) return;
    const int64_t step = (int64_t)nwarps * rpw;
    for (int64_t t = t0 + warp * rpw + r; t < t1; t += step * U) {
      float v[U];
#pragma unroll
      for (int u = 0; u < U; ++u)
        if (t + u * step < t1) v[u] = S[(t + u * step) * E + c0 + cc];
#pragma unroll
      for (int u = 0; u < U; ++u)
        if (t + u * step < t1) f(v[u], t + u * step, 0);
    }
  }
}

template <bool VEC>
__global__ void __launch_bounds__(kHistThreads, 1)
topk_hist_kernel(const float* __restrict__ S, int64_t n, int E, unsigned k, int pass, int rows_per_cta,
                 SelState* state, unsigned* hist, unsigned* counters) {
  extern __shared__ unsigned sh[];                     // [bin][column]
  __shared__ unsigned long long s_prefix[kTopkChunk];
  __shared__ int s_active[kTopkChunk];
  __shared__ int s_any, s_last;
  const int tid = threadIdx.x, chunk = blockIdx.y, nchunks = gridDim.y, grp = blockIdx.z;
  const int c0 = chunk * kTopkChunk, cw = min(kTopkChunk, E - c0);
  S += (size_t)grp * n * E;                            // this group's n rows; its experts' state, histograms
  state += (size_t)grp * E; hist += (size_t)grp * E * kBins; counters += (size_t)grp * kRadixPasses * nchunks;
  if (tid == 0) s_any = 0;
  __syncthreads();
  if (tid < kTopkChunk) {
    int act = 0; unsigned long long pre = 0;
    if (tid < cw) {
      if (pass == 0) act = 1;
      else { act = state[c0 + tid].mode == 0 ? 1 : 0; pre = state[c0 + tid].prefix; }
    }
    s_active[tid] = act; s_prefix[tid] = pre;
    if (act) s_any = 1;
  }
  for (int i = tid; i < kBins * kTopkChunk; i += kHistThreads) sh[i] = 0;
  __syncthreads();
  if (!s_any) return;                                  // uniform: every expert of the chunk is decided
  const int shift = 52 - kRadixBits * pass;            // score bits 29..20, 19..10, 9..0
  const int64_t t0 = (int64_t)blockIdx.x * rows_per_cta;
  const int64_t t1 = min(n, t0 + rows_per_cta);
  {
    // only the score half of the key matters here: v = ~bits(S), digit (v >> sh32) & 1023, and from the
    // second pass on the bits above the digit have to equal the expert's prefix
    constexpr int NC = VEC ? 4 : 1;
    const int col0 = slab_first_col<VEC>(cw), sh32 = shift - 32;
    bool act[NC]; unsigned want[NC];
#pragma unroll
    for (int j = 0; j < NC; ++j) {
      act[j] = col0 >= 0 && col0 + j < cw && s_active[col0 + j];
      want[j] = act[j] ? (unsigned)(s_prefix[col0 + j] >> 32) >> (sh32 + kRadixBits) : 0u;
    }
    for_slab<VEC>(S, E, c0, cw, t0, t1, [&](float s, int64_t, int j) {
      const unsigned v = ~__float_as_uint(s);
      if (act[j] && (pass == 0 || (v >> (sh32 + kRadixBits)) == want[j]))
        atomicAdd(&sh[((v >> sh32) & (kBins - 1)) * kTopkChunk + col0 + j], 1u);
    });
  }
  __syncthreads();
  for (int i = tid; i < kBins * kTopkChunk; i += kHistThreads) {
    const unsigned v = sh[i];
    if (v) atomicAdd(&hist[(size_t)(c0 + i % kTopkChunk) * kBins + i / kTopkChunk], v);
  }
  __threadfence();
  __syncthreads();
  if (tid == 0) s_last = atomicAdd(&counters[pass * nchunks + chunk], 1u) == gridDim.x - 1;
  __syncthreads();
  if (!s_last) return;
  __threadfence();
  // The last CTA of this chunk sees the full histograms: one warp per expert finds the bucket of the
  // k-th key, records the decision and leaves the histogram zeroed for the next pass.
  const int warp = tid >> 5, lane = tid & 31;
  if (warp >= cw || !s_active[warp]) return;
  // The expert's kBins counts come in with coalesced, independent loads (lane holds bins lane, 32 + lane, ...),
  // are laid out in the CTA's shared histogram (free by now; one padding word per 32 keeps the banks
  // apart) and are read back as 32 consecutive bins per lane.
  unsigned* h = hist + (size_t)(c0 + warp) * kBins;
  constexpr int PER = kBins / 32;
  unsigned* col = sh + warp * (kBins + PER);
  {
    unsigned tmp[PER];
#pragma unroll
    for (int j = 0; j < PER; ++j) tmp[j] = __ldcg(h + j * 32 + lane);
#pragma unroll
    for (int j = 0; j < PER; ++j) { h[j * 32 + lane] = 0; col[j * 33 + lane] = tmp[j]; }
  }
  __syncwarp();
  unsigned lsum = 0;
#pragma unroll
  for (int j = 0; j < PER; ++j) lsum += col[lane * 33 + j];
  unsigned incl = lsum;
  for (int o = 1; o < 32; o <<= 1) { const unsigned v = __shfl_up_sync(0xffffffffu, incl, o); if (lane >= o) incl += v; }
  const unsigned excl = incl - lsum;
  const unsigned k_rem = pass == 0 ? k : state[c0 + warp].k_rem;
  if (excl < k_rem && k_rem <= incl) {                 // exactly one lane
    unsigned before = excl, in_bucket = 0; int D = 0;
    for (int j = 0; j < PER; ++j) {
      const unsigned c = col[lane * 33 + j];
      if (k_rem <= before + c) { D = j; in_bucket = c; break; }
      before += c;
    }
    const unsigned new_rem = k_rem - before;
    SelState ns;
    ns.prefix = (pass == 0 ? kKeyTop : s_prefix[warp]) | ((unsigned long long)(lane * PER + D) << shift);
    ns.shift = (unsigned)shift; ns.k_rem = new_rem; ns.cand = 0;
    if (in_bucket == new_rem) ns.mode = 1;                             // the whole bucket is taken
    else if (in_bucket <= (unsigned)kCandCap) { ns.mode = 2; ns.cand = in_bucket; }   // the sort picks new_rem of these
    else ns.mode = 0;                                                  // descend one more digit
    state[c0 + warp] = ns;
  }
}

// Experts undecided after the score passes: more than kCandCap keys share the threshold score exactly,
// and the k_rem lowest tokens among them win.  One CTA per expert walks the column in token order.
__global__ void __launch_bounds__(1024)
topk_ties_kernel(const float* __restrict__ S, int64_t n, int E, unsigned k, int64_t kpad, SelState* state,
                 unsigned long long* keys) {
  __shared__ unsigned s_warp[32];
  __shared__ unsigned s_total;
  const int e = blockIdx.x, grp = blockIdx.y, tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  S += (size_t)grp * n * E; state += (size_t)grp * E; keys += (size_t)grp * E * kpad;
  if (state[e].mode != 0) return;
  const unsigned thr = (unsigned)(state[e].prefix >> 32), k_rem = state[e].k_rem, k_def = k - k_rem;
  unsigned running = 0;
  for (int64_t base = 0; base < n && running < k_rem; base += 1024) {
    const int64_t t = base + tid;
    float s = 0.f; bool m = false;
    if (t < n) { s = S[t * E + e]; m = ~__float_as_uint(s) == thr; }
    const unsigned bal = __ballot_sync(0xffffffffu, m);
    if (lane == 0) s_warp[warp] = __popc(bal);
    __syncthreads();
    if (warp == 0) {
      const unsigned v = s_warp[lane];
      unsigned inc = v;
      for (int o = 1; o < 32; o <<= 1) { const unsigned u = __shfl_up_sync(0xffffffffu, inc, o); if (lane >= o) inc += u; }
      s_warp[lane] = inc - v;
      if (lane == 31) s_total = inc;
    }
    __syncthreads();
    const unsigned idx = running + s_warp[warp] + __popc(bal & ((1u << lane) - 1u));
    if (m && idx < k_rem) keys[(size_t)e * kpad + k_def + idx] = make_key(s, t);
    running += s_total;
    __syncthreads();
  }
  if (tid == 0) state[e].mode = 3;
}

// Copies each expert's winners to keys[i][0 ..) and its candidates to cand[i][0 ..), in no particular
// order, with one read of S: a CTA parks what it finds in shared memory, reserves one range per
// (expert, kind) with a single global atomic each and writes the keys out.  What does not fit in the
// buffer (only with very uneven inputs) takes its place with a global atomic of its own.
constexpr int kCompactCap = 4096;
template <bool VEC>
__global__ void __launch_bounds__(kHistThreads)
topk_compact_kernel(const float* __restrict__ S, int64_t n, int E, unsigned k, int64_t kpad, int rows_per_cta,
                    const SelState* __restrict__ state, unsigned* cursor, unsigned long long* keys,
                    unsigned long long* cand) {
  __shared__ unsigned long long s_key[kCompactCap];
  __shared__ unsigned char s_tag[kCompactCap];         // column within the chunk, bit 7: candidate
  __shared__ unsigned s_cnt[2][kTopkChunk], s_base[2][kTopkChunk], s_n;
  __shared__ unsigned long long s_thr[kTopkChunk];
  __shared__ unsigned s_shift[kTopkChunk], s_mode[kTopkChunk];
  const int tid = threadIdx.x, chunk = blockIdx.y, grp = blockIdx.z, groups = gridDim.z;
  const int c0 = chunk * kTopkChunk, cw = min(kTopkChunk, E - c0);
  S += (size_t)grp * n * E; state += (size_t)grp * E;
  keys += (size_t)grp * E * kpad; cand += (size_t)grp * E * kCandCap;
  unsigned* cursor_w = cursor + (size_t)grp * E;                       // winners; candidates follow all groups' winners
  unsigned* cursor_c = cursor + (size_t)groups * E + (size_t)grp * E;
  if (tid == 0) s_n = 0;
  if (tid < kTopkChunk) {
    s_cnt[0][tid] = s_cnt[1][tid] = 0;
    if (tid < cw) {
      const SelState st = state[c0 + tid];
      s_shift[tid] = st.shift; s_thr[tid] = st.prefix >> st.shift; s_mode[tid] = st.mode;
    }
  }
  __syncthreads();
  const int64_t t0 = (int64_t)blockIdx.x * rows_per_cta;
  const int64_t t1 = min(n, t0 + rows_per_cta);
  auto put = [&](int kind, int col, unsigned pos, unsigned long long key) {      // kind 0: winner, 1: candidate
    if (kind == 0) { if (pos < k) keys[(size_t)(c0 + col) * kpad + pos] = key; }
    else if (pos < (unsigned)kCandCap) cand[(size_t)(c0 + col) * kCandCap + pos] = key;
  };
  // per column of this thread: the decided score bits (thr, after dropping the low bits of v = ~bits(S) that
  // are still open) and what happens to a key exactly at the threshold: 0 winner, 1 candidate, 2 nothing
  // (the tie walk has placed it)
  constexpr int NC = VEC ? 4 : 1;
  const int col0 = slab_first_col<VEC>(cw);
  unsigned thr[NC], drop[NC]; int at_thr[NC];
#pragma unroll
  for (int j = 0; j < NC; ++j) {
    const bool ok = col0 >= 0 && col0 + j < cw;
    drop[j] = ok ? s_shift[col0 + j] - 32 : 0; thr[j] = ok ? (unsigned)s_thr[col0 + j] : 0u;
    at_thr[j] = !ok ? 2 : (s_mode[col0 + j] == 1 ? 0 : (s_mode[col0 + j] == 2 ? 1 : 2));
  }
  for_slab<VEC>(S, E, c0, cw, t0, t1, [&](float s, int64_t t, int j) {
    const unsigned hi = ~__float_as_uint(s) >> drop[j];
    if (hi > thr[j]) return;
    const int kind = hi < thr[j] ? 0 : at_thr[j];
    if (kind == 2) return;
    const int col = col0 + j;
    const unsigned long long key = make_key(s, t);
    const unsigned idx = atomicAdd(&s_n, 1u);
    if (idx < (unsigned)kCompactCap) { s_key[idx] = key; s_tag[idx] = (unsigned char)(col | (kind << 7)); }
    else put(kind, col, atomicAdd(&(kind ? cursor_c : cursor_w)[c0 + col], 1u), key);
  });
  __syncthreads();
  const int held = (int)min(s_n, (unsigned)kCompactCap);
  for (int i = tid; i < held; i += kHistThreads) atomicAdd(&s_cnt[s_tag[i] >> 7][s_tag[i] & 127], 1u);
  __syncthreads();
  if (tid < 2 * kTopkChunk) {
    const int w = tid / kTopkChunk, col = tid % kTopkChunk;
    if (col < cw) { const unsigned c = s_cnt[w][col]; s_base[w][col] = c ? atomicAdd(&(w ? cursor_c : cursor_w)[c0 + col], c) : 0u; }
  }
  __syncthreads();
  if (tid < kTopkChunk) s_cnt[0][tid] = s_cnt[1][tid] = 0;
  __syncthreads();
  for (int i = tid; i < held; i += kHistThreads) {
    const int kind = s_tag[i] >> 7, col = s_tag[i] & 127;
    put(kind, col, s_base[kind][col] + atomicAdd(&s_cnt[kind][col], 1u), s_key[i]);
  }
}

// Slot j of virtual expert ve = group * E + expert lands in row `expert` of I and G (each groups * k long) at
// position group * k + j, and the token index becomes global (group * n + token within the group).
struct SlotMap { int E, groups; int64_t k, n; };
__device__ __forceinline__ void emit_slot(unsigned long long key, int32_t* I, float* G, const SlotMap& m, int64_t ve, int64_t j) {
  const int64_t grp = ve / m.E, e = ve % m.E;
  const int64_t o = (e * m.groups + grp) * m.k + j;
  I[o] = (int32_t)((unsigned)(key & 0xFFFFFFFFull) + (unsigned)(grp * m.n));
  G[o] = __uint_as_float(~(unsigned)(key >> 32));
}

// Ascending bitonic sort of len (a power of two) keys in shared memory by the whole CTA.
__device__ __forceinline__ void bitonic_smem(unsigned long long* a, int len) {
  for (int size = 2; size <= len; size <<= 1) {
    for (int stride = size >> 1; stride >= 1; stride >>= 1) {
      for (int p = threadIdx.x; p < (len >> 1); p += blockDim.x) {
        const int i = ((p & ~(stride - 1)) << 1) | (p & (stride - 1)), j = i + stride;      // stride is a power of two
        const bool asc = (i & size) == 0;
        const unsigned long long x = a[i], y = a[j];
        if ((x > y) == asc) { a[i] = y; a[j] = x; }
      }
      __syncthreads();
    }
  }
}

// Sorts an expert's candidates and returns (in shared memory) them in ascending order; sc holds kCandCap keys.
__device__ __forceinline__ void load_sorted_candidates(const unsigned long long* cand, int e, unsigned ncand,
                                                       unsigned long long* sc) {
  const int len = pow2_at_least((int)ncand);
  for (int i = threadIdx.x; i < len; i += blockDim.x) sc[i] = i < (int)ncand ? cand[(size_t)e * kCandCap + i] : ~0ull;
  __syncthreads();
  bitonic_smem(sc, len);
}

// k up to one tile: one CTA per expert merges the candidates in, sorts the k keys and writes I and G.
constexpr int kSortThreads = 1024;
__global__ void __launch_bounds__(kSortThreads)
topk_finish_tile_kernel(const unsigned long long* __restrict__ keys, const unsigned long long* __restrict__ cand,
                        const SelState* __restrict__ state, int64_t kpad, int64_t k, SlotMap map, int32_t* I, float* G) {
  __shared__ unsigned long long sk[kSortTile];
  __shared__ unsigned long long sc[kCandCap];
  const int e = blockIdx.x;
  const SelState st = state[e];
  for (int i = threadIdx.x; i < kpad; i += kSortThreads) sk[i] = keys[(size_t)e * kpad + i];
  __syncthreads();
  if (st.mode == 2) {
    load_sorted_candidates(cand, e, st.cand, sc);
    const unsigned k_def = (unsigned)k - st.k_rem;
    for (int i = threadIdx.x; i < (int)st.k_rem; i += kSortThreads) sk[k_def + i] = sc[i];
    __syncthreads();
  }
  bitonic_smem(sk, (int)kpad);
  for (int i = threadIdx.x; i < k; i += kSortThreads) emit_slot(sk[i], I, G, map, e, i);
}

// k beyond one tile: the candidates are merged into the global key list first.
__global__ void __launch_bounds__(kSortThreads)
topk_resolve_kernel(unsigned long long* keys, const unsigned long long* __restrict__ cand,
                    const SelState* __restrict__ state, int64_t kpad, int64_t k) {
  __shared__ unsigned long long sc[kCandCap];
  const int e = blockIdx.x;
  const SelState st = state[e];
  if (st.mode != 2) return;
  load_sorted_candidates(cand, e, st.cand, sc);
  const unsigned k_def = (unsigned)k - st.k_rem;
  for (int i = threadIdx.x; i < (int)st.k_rem; i += kSortThreads) keys[(size_t)e * kpad + k_def + i] = sc[i];
}

// Bitonic steps on one tile of kSortTile keys held in shared memory.  Runs the network sizes
// size_lo..size_hi (powers of two); for a size larger than the tile only the strides that fit.
__global__ void __launch_bounds__(kSortThreads)
topk_sort_tile_kernel(unsigned long long* keys, int64_t kpad, int64_t k, int64_t size_lo, int64_t size_hi,
                      int emit, SlotMap map, int32_t* I, float* G) {
  __shared__ unsigned long long sk[kSortTile];
  const int64_t tiles_per_expert = (kpad + kSortTile - 1) / kSortTile;
  const int64_t expert = blockIdx.x / tiles_per_expert;
  const int64_t base = (blockIdx.x % tiles_per_expert) * kSortTile;   // index inside the expert
  const int len = (int)min((int64_t)kSortTile, kpad - base);          // power of two
  unsigned long long* src = keys + expert * kpad + base;
  for (int i = threadIdx.x; i < len; i += kSortThreads) sk[i] = src[i];
  __syncthreads();
  for (int64_t size = size_lo; size <= size_hi; size <<= 1) {
    for (int64_t stride = min(size >> 1, (int64_t)(len >> 1)); stride >= 1; stride >>= 1) {
      for (int p = threadIdx.x; p < (len >> 1); p += kSortThreads) {
        const int i = (int)((((int64_t)p & ~(stride - 1)) << 1) | ((int64_t)p & (stride - 1)));   // stride is a power of two
        const int j = i + (int)stride;
        const bool asc = ((base + i) & size) == 0;
        const unsigned long long a = sk[i], b = sk[j];
        if ((a > b) == asc) { sk[i] = b; sk[j] = a; }
      }
      __syncthreads();
    }
  }
  if (emit) {
    for (int i = threadIdx.x; i < len; i += kSortThreads)
      if (base + i < k) emit_slot(sk[i], I, G, map, expert, base + i);
  } else {
    for (int i = threadIdx.x; i < len; i += kSortThreads) src[i] = sk[i];
  }
}

// One compare-exchange step at a stride that spans tiles.
__global__ void topk_sort_global_kernel(unsigned long long* keys, int64_t kpad, int64_t total_pairs,
                                        int64_t size, int64_t stride) {
  for (int64_t p = (int64_t)blockIdx.x * blockDim.x + threadIdx.x; p < total_pairs;
       p += (int64_t)gridDim.x * blockDim.x) {
    const int64_t expert = p / (kpad >> 1), q = p % (kpad >> 1);
    const int64_t i = ((q & ~(stride - 1)) << 1) | (q & (stride - 1)), j = i + stride;       // stride is a power of two
    unsigned long long* kk = keys + expert * kpad;
    const bool asc = (i & size) == 0;
    const unsigned long long a = kk[i], b = kk[j];
    if ((a > b) == asc) { kk[i] = b; kk[j] = a; }
  }
}

// Small groups (n <= kSmallN tokens, k <= kSortTile): the whole selection of one expert in one CTA.  The
// column is brought into shared memory once (as v = ~bits(S)), three 10-bit histogram passes over it find
// the value of the k-th key exactly, keys below it are winners, keys equal to it win in token order, and the
// k keys are sorted and written out: one launch instead of eight, for the sizes where launches are what costs.
constexpr int kSmallN = 16384;
__global__ void __launch_bounds__(1024)
topk_small_kernel(const float* __restrict__ S, int n, int E, int k, int kpad, SlotMap map, int32_t* I, float* G) {
  extern __shared__ unsigned long long sm_keys[];      // [kpad] keys, then [n] values, then [kBins] histogram
  unsigned* val = reinterpret_cast<unsigned*>(sm_keys + kpad);
  unsigned* hist = val + n;
  __shared__ unsigned s_prefix, s_rem, s_less, s_eqtaken, s_warp[33];
  const int e = blockIdx.x, grp = blockIdx.y, tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const int nt = blockDim.x, nwarps = nt >> 5;         // 128 .. 1024 threads, by the size of the group
  const float* col = S + (size_t)grp * n * E + e;
  for (int t = tid; t < n; t += nt) val[t] = ~__float_as_uint(col[(size_t)t * E]);
  for (int i = tid; i < kpad; i += nt) sm_keys[i] = ~0ull;
  if (tid == 0) { s_prefix = 0; s_rem = (unsigned)k; s_less = 0; s_eqtaken = 0; }
  __syncthreads();
  // v has its two top bits set (0 <= S <= 1); digits of 10 bits from bit 29 down
  for (int pass = 0; pass < 3; ++pass) {
    const int sh = 20 - 10 * pass;
    for (int i = tid; i < kBins; i += nt) hist[i] = 0;
    __syncthreads();
    const unsigned pre = s_prefix;
    for (int t = tid; t < n; t += nt) {
      const unsigned v = val[t];
      if (pass == 0 || (v >> (sh + 10)) == (pre >> (sh + 10))) atomicAdd(&hist[(v >> sh) & (kBins - 1)], 1u);
    }
    __syncthreads();
    if (warp == 0) {                                   // bucket of the s_rem-th smallest v among the matching ones
      unsigned c[kBins / 32], lsum = 0;
#pragma unroll
      for (int j = 0; j < kBins / 32; ++j) { c[j] = hist[lane * (kBins / 32) + j]; lsum += c[j]; }
      unsigned incl = lsum;
      for (int o = 1; o < 32; o <<= 1) { const unsigned u = __shfl_up_sync(0xffffffffu, incl, o); if (lane >= o) incl += u; }
      const unsigned excl = incl - lsum, rem = s_rem;
      if (excl < rem && rem <= incl) {
        unsigned before = excl; int D = 0;
#pragma unroll
        for (int j = 0; j < kBins / 32; ++j) {
          if (before < rem && rem <= before + c[j]) { D = j; break; }
          before += c[j];
        }
        s_prefix = (pass == 0 ? 0xC0000000u : pre) | ((unsigned)(lane * (kBins / 32) + D) << sh);
        s_rem = rem - before;
      }
    }
    __syncthreads();
  }
  const unsigned thr = s_prefix, k_rem = s_rem, k_less = (unsigned)k - k_rem;      // k_rem keys equal to thr are wanted
  // winners strictly below the threshold: any order
  for (int t = tid; t < n; t += nt)
    if (val[t] < thr) sm_keys[atomicAdd(&s_less, 1u)] = ((unsigned long long)val[t] << 32) | (unsigned)t;
  // keys at the threshold: the first k_rem in token order
  unsigned running = 0;
  for (int base = 0; base < n && running < k_rem; base += nt) {
    const int t = base + tid;
    const bool m = t < n && val[t] == thr;
    const unsigned bal = __ballot_sync(0xffffffffu, m);
    if (lane == 0) s_warp[warp] = __popc(bal);
    __syncthreads();
    if (warp == 0) {
      const unsigned v = lane < nwarps ? s_warp[lane] : 0u;
      unsigned inc = v;
      for (int o = 1; o < 32; o <<= 1) { const unsigned u = __shfl_up_sync(0xffffffffu, inc, o); if (lane >= o) inc += u; }
      s_warp[lane] = inc - v;
      if (lane == 31) s_warp[32] = inc;
    }
    __syncthreads();
    const unsigned idx = running + s_warp[warp] + __popc(bal & ((1u << lane) - 1u));
    if (m && idx < k_rem) sm_keys[k_less + idx] = ((unsigned long long)thr << 32) | (unsigned)t;
    running += s_warp[32];
    __syncthreads();
  }
  __syncthreads();
  bitonic_smem(sm_keys, kpad);
  for (int i = tid; i < k; i += nt) emit_slot(sm_keys[i], I, G, map, (int64_t)grp * E + e, i);
}

cudaError_t launch_topk(const float* S, int64_t n, int E, int64_t k, int groups, int32_t* I, float* G,
                        void* scratch, cudaStream_t st) {
  const TopkLayout L = topk_layout(n, E, k, groups);
  if (n <= kSmallN && L.kpad <= kSortTile) {
    const SlotMap smap = {E, groups, k, n};
    const int smem = (int)(L.kpad * 8 + n * 4 + kBins * 4);
    cudaError_t e0 = cudaFuncSetAttribute(topk_small_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, smem);
    if (e0 != cudaSuccess) return e0;
    int threads = 128;                                 // about eight elements per thread
    while (threads < 1024 && threads * 8 < n) threads <<= 1;
    count_launch();
    topk_small_kernel<<<dim3(E, groups), threads, smem, st>>>(S, (int)n, E, (int)k, (int)L.kpad, smap, I, G);
    return cudaGetLastError();
  }
  const int64_t VE = (int64_t)groups * E;              // independent columns: E per group
  char* base = (char*)scratch;
  SelState* state = (SelState*)(base + L.off_state);
  unsigned* hist = (unsigned*)(base + L.off_hist);
  unsigned* counters = (unsigned*)(base + L.off_counters);
  unsigned* cursor = (unsigned*)(base + L.off_cursor);
  unsigned long long* cand = (unsigned long long*)(base + L.off_cand);
  unsigned long long* keys = (unsigned long long*)(base + L.off_keys);
  const SlotMap map = {E, groups, k, n};
  cudaError_t e;
  const bool vec = E % 4 == 0 && ((uintptr_t)S & 15) == 0;
  // the histogram kernels use 132 KiB of dynamic shared memory
  if ((e = vec ? cudaFuncSetAttribute(topk_hist_kernel<true>, cudaFuncAttributeMaxDynamicSharedMemorySize, kHistSmemBytes)
               : cudaFuncSetAttribute(topk_hist_kernel<false>, cudaFuncAttributeMaxDynamicSharedMemorySize, kHistSmemBytes)) != cudaSuccess) return e;
  if ((e = cudaMemsetAsync(base, 0, L.zero_bytes, st)) != cudaSuccess) return e;
  if ((e = cudaMemsetAsync(keys, 0xFF, (size_t)VE * L.kpad * 8, st)) != cudaSuccess) return e;
  // rows per CTA: one CTA per SM fits (the histogram takes 132 KiB of shared memory), so one wave over all
  // chunks and groups; at least 256 rows each
  int64_t want = (int64_t)148 / ((int64_t)L.chunks * groups); if (want < 1) want = 1;
  int64_t rows = (n + want - 1) / want; if (rows < 256) rows = 256;
  const dim3 grid((unsigned)((n + rows - 1) / rows), (unsigned)L.chunks, (unsigned)groups);
  for (int pass = 0; pass < kRadixPasses; ++pass) {
    count_launch();
    if (vec) topk_hist_kernel<true><<<grid, kHistThreads, kHistSmemBytes, st>>>(S, n, E, (unsigned)k, pass, (int)rows, state, hist, counters);
    else topk_hist_kernel<false><<<grid, kHistThreads, kHistSmemBytes, st>>>(S, n, E, (unsigned)k, pass, (int)rows, state, hist, counters);
  }
  count_launch();
  topk_ties_kernel<<<dim3(E, groups), 1024, 0, st>>>(S, n, E, (unsigned)k, L.kpad, state, keys);
  count_launch();
  if (vec) topk_compact_kernel<true><<<grid, kHistThreads, 0, st>>>(S, n, E, (unsigned)k, L.kpad, (int)rows, state, cursor, keys, cand);
  else topk_compact_kernel<false><<<grid, kHistThreads, 0, st>>>(S, n, E, (unsigned)k, L.kpad, (int)rows, state, cursor, keys, cand);
  if (L.kpad <= kSortTile) {
    count_launch();
    topk_finish_tile_kernel<<<(unsigned)VE, kSortThreads, 0, st>>>(keys, cand, state, L.kpad, k, map, I, G);
  } else {
    const int64_t tiles = (L.kpad + kSortTile - 1) / kSortTile;
    const unsigned sort_grid = (unsigned)(VE * tiles);
    count_launch();
    topk_resolve_kernel<<<(unsigned)VE, kSortThreads, 0, st>>>(keys, cand, state, L.kpad, k);
    count_launch();
    topk_sort_tile_kernel<<<sort_grid, kSortThreads, 0, st>>>(keys, L.kpad, k, 2, kSortTile, 0, map, I, G);
    const int64_t pairs = VE * (L.kpad >> 1);
    for (int64_t size = 2 * kSortTile; size <= L.kpad; size <<= 1) {
      for (int64_t stride = size >> 1; stride >= kSortTile; stride >>= 1) {
        count_launch();
        topk_sort_global_kernel<<<grid_for(pairs, 256), 256, 0, st>>>(keys, L.kpad, pairs, size, stride);
      }
      count_launch();
      topk_sort_tile_kernel<<<sort_grid, kSortThreads, 0, st>>>(keys, L.kpad, k, size, size, size == L.kpad, map, I, G);
    }
  }
  return cudaGetLastError();
}

// ------------------------------------------------------------------------------------------
// Token-choice contrast routing (Section 3.1): every token picks its two best experts, experts have buffers.
// ------------------------------------------------------------------------------------------
// One warp per token row of S: the two largest scores, equal scores to the lower expert.  A score in [0, 1] orders
// like its bit pattern; the key puts the inverted expert index below it so that one max decides both.
__global__ void __launch_bounds__(256) token_top2_kernel(const float* __restrict__ S, int64_t rows, int E, int32_t* __restrict__ choice) {
  const int lane = threadIdx.x & 31;
  const int64_t warps = ((int64_t)gridDim.x * blockDim.x) >> 5;
  for (int64_t t = ((int64_t)blockIdx.x * blockDim.x + threadIdx.x) >> 5; t < rows; t += warps) {
    unsigned long long best = 0, second = 0;           // 0 is below every real key (the index part of a real key is > 0)
    for (int i = lane; i < E; i += 32) {
      const unsigned long long key = ((unsigned long long)__float_as_uint(S[t * E + i]) << 32) | (0xFFFFFFFFu - (unsigned)i);
      if (key > best) { second = best; best = key; } else if (key > second) second = key;
    }
    unsigned long long top = best;
    for (int o = 16; o; o >>= 1) { const unsigned long long v = __shfl_xor_sync(0xffffffffu, top, o); top = v > top ? v : top; }
    const unsigned long long mine = best == top ? second : best;          // the winner's lane offers its runner-up
    unsigned long long nxt = mine;
    for (int o = 16; o; o >>= 1) { const unsigned long long v = __shfl_xor_sync(0xffffffffu, nxt, o); nxt = v > nxt ? v : nxt; }
    if (lane == 0) {
      choice[2 * t] = (int32_t)(0xFFFFFFFFu - (unsigned)top);
      choice[2 * t + 1] = (int32_t)(0xFFFFFFFFu - (unsigned)nxt);
    }
  }
}

// One CTA per (expert, group) walks the group's tokens in order; a token that chose the expert takes the next slot
// while there is one.  A token's two choices are different experts, so the order of the requests to one expert is
// the token order.  Empty slots get -1 / 0.
__global__ void __launch_bounds__(1024)
token_admit_kernel(const float* __restrict__ S, const int32_t* __restrict__ choice, int n, int E, int k,
                   int32_t* __restrict__ I, float* __restrict__ G, int32_t* __restrict__ load, int32_t* __restrict__ requested) {
  __shared__ unsigned s_warp[33];
  const int e = blockIdx.x, grp = blockIdx.y, groups = gridDim.y, tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  const int64_t row0 = (int64_t)grp * n;
  int32_t* Ie = I + ((int64_t)e * groups + grp) * k;
  float* Ge = G + ((int64_t)e * groups + grp) * k;
  unsigned running = 0;
  for (int base = 0; base < n; base += 1024) {
    const int t = base + tid;
    bool m = false;
    if (t < n) { const int2 c = *reinterpret_cast<const int2*>(choice + 2 * (row0 + t)); m = c.x == e || c.y == e; }
    const unsigned bal = __ballot_sync(0xffffffffu, m);
    if (lane == 0) s_warp[warp] = __popc(bal);
    __syncthreads();
    if (warp == 0) {
      const unsigned v = s_warp[lane];
      unsigned inc = v;
      for (int o = 1; o < 32; o <<= 1) { const unsigned u = __shfl_up_sync(0xffffffffu, inc, o); if (lane >= o) inc += u; }
      s_warp[lane] = inc - v;
      if (lane == 31) s_warp[32] = inc;
    }
    __syncthreads();
    const unsigned pos = running + s_warp[warp] + __popc(bal & ((1u << lane) - 1u));
    if (m && pos < (unsigned)k) { Ie[pos] = (int32_t)(row0 + t); Ge[pos] = S[(row0 + t) * E + e]; }
    running += s_warp[32];
    __syncthreads();
  }
  const unsigned filled = running < (unsigned)k ? running : (unsigned)k;
  for (int j = (int)filled + tid; j < k; j += 1024) { Ie[j] = -1; Ge[j] = 0.f; }
  if (tid == 0) { load[grp * E + e] = (int32_t)filled; requested[grp * E + e] = (int32_t)running; }
}

cudaError_t launch_token_top2(const float* S, int64_t rows, int E, int32_t* choice, cudaStream_t st) {
  count_launch();
  token_top2_kernel<<<grid_for(rows * 32, 256, 148 * 8), 256, 0, st>>>(S, rows, E, choice);
  return cudaGetLastError();
}

cudaError_t launch_token_admit(const float* S, const int32_t* choice, int64_t n, int E, int64_t k, int groups,
                               int32_t* I, float* G, int32_t* load, int32_t* requested, cudaStream_t st) {
  count_launch();
  token_admit_kernel<<<dim3(E, groups), 1024, 0, st>>>(S, choice, (int)n, E, (int)k, I, G, load, requested);
  return cudaGetLastError();
}

// ------------------------------------------------------------------------------------------
// Index form of P = Onehot(I) (Eq. 2) read by token: row_ptr / slots.
// Integer atomics only count and hand out positions; each token's short list is then sorted,
// so the result does not depend on the order in which threads ran.
// scratch: [cnt n+1 int32][tile sums ceil(n / kScanTile) int32]
// ------------------------------------------------------------------------------------------
constexpr int kScanTile = 4096, kScanThreads = 1024;
static size_t inv_cnt_bytes(int64_t n) { return ((size_t)(n + 1) * 4 + 255) & ~(size_t)255; }
size_t inverse_scratch_bytes(int64_t n) {
  return inv_cnt_bytes(n) + ((((size_t)(n + kScanTile - 1) / kScanTile) * 4 + 255) & ~(size_t)255);
}

__global__ void inv_count_kernel(const int32_t* __restrict__ I, int64_t total, int32_t* cnt, int64_t n, int* status) {
  for (int64_t s = (int64_t)blockIdx.x * blockDim.x + threadIdx.x; s < total; s += (int64_t)gridDim.x * blockDim.x) {
    const int t = I[s];
    if (t >= 0 && idx_ok(t, 0, n, status)) atomicAdd(&cnt[t], 1);      // -1: an empty slot (token-choice routing only)
  }
}

// Exclusive scan of the CTA's per-thread values (any thread count that is a multiple of 32, at most 1024);
// returns the thread's offset and, in `total`, the sum over the CTA.
__device__ __forceinline__ int block_exclusive_scan(int v, int* s_warp, int& total) {
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5, nwarps = blockDim.x >> 5;
  int inc = v;
  for (int o = 1; o < 32; o <<= 1) { const int u = __shfl_up_sync(0xffffffffu, inc, o); if (lane >= o) inc += u; }
  if (lane == 31) s_warp[warp] = inc;
  __syncthreads();
  if (warp == 0) {
    const int w = lane < nwarps ? s_warp[lane] : 0;
    int winc = w;
    for (int o = 1; o < 32; o <<= 1) { const int u = __shfl_up_sync(0xffffffffu, winc, o); if (lane >= o) winc += u; }
    s_warp[lane] = winc - w;
    if (lane == 31) s_warp[32] = winc;
  }
  __syncthreads();
  total = s_warp[32];
  return s_warp[warp] + inc - v;
}

// Step 1: exclusive scan inside each tile of kScanTile counts (four per thread), tile sums aside.
__global__ void __launch_bounds__(kScanThreads) inv_scan_tile_kernel(const int32_t* __restrict__ cnt, int64_t n,
                                                                      int32_t* row_ptr, int32_t* tile_sum) {
  __shared__ int s_warp[33];
  const int64_t base = (int64_t)blockIdx.x * kScanTile + threadIdx.x * 4;
  int c[4];
#pragma unroll
  for (int j = 0; j < 4; ++j) c[j] = base + j < n ? cnt[base + j] : 0;
  int total;
  int run = block_exclusive_scan(c[0] + c[1] + c[2] + c[3], s_warp, total);
#pragma unroll
  for (int j = 0; j < 4; ++j) { if (base + j < n) row_ptr[base + j] = run; run += c[j]; }
  if (threadIdx.x == 0) tile_sum[blockIdx.x] = total;
}

// Step 2: every tile adds the sum of the tiles before it; the last one also writes row_ptr[n].
__global__ void __launch_bounds__(kScanThreads) inv_scan_add_kernel(const int32_t* __restrict__ tile_sum, int64_t n,
                                                                     int32_t* row_ptr) {
  __shared__ int s_warp[33];
  int part = 0;
  for (int j = threadIdx.x; j < (int)blockIdx.x; j += kScanThreads) part += tile_sum[j];
  int before;
  block_exclusive_scan(part, s_warp, before);
  const int64_t base = (int64_t)blockIdx.x * kScanTile + threadIdx.x * 4;
#pragma unroll
  for (int j = 0; j < 4; ++j) if (base + j < n) row_ptr[base + j] += before;
  if (blockIdx.x == gridDim.x - 1 && threadIdx.x == 0) row_ptr[n] = before + tile_sum[blockIdx.x];
}

// Hands each slot a place in its token's list, counting the token's counter back down to zero.
__global__ void inv_fill_kernel(const int32_t* __restrict__ I, int64_t total, const int32_t* __restrict__ row_ptr,
                                int32_t* cnt, int32_t* slots, int64_t n) {
  for (int64_t s = (int64_t)blockIdx.x * blockDim.x + threadIdx.x; s < total; s += (int64_t)gridDim.x * blockDim.x) {
    const int t = I[s];
    if (t >= 0 && idx_ok(t, 0, n, nullptr)) slots[row_ptr[t] + atomicSub(&cnt[t], 1) - 1] = (int32_t)s;   // counted once, in inv_count
  }
}

__global__ void inv_sort_kernel(const int32_t* __restrict__ row_ptr, int64_t n, int32_t* slots) {
  for (int64_t t = (int64_t)blockIdx.x * blockDim.x + threadIdx.x; t < n; t += (int64_t)gridDim.x * blockDim.x) {
    const int a = row_ptr[t], b = row_ptr[t + 1];
    for (int i = a + 1; i < b; ++i) {
      const int v = slots[i]; int j = i - 1;
      while (j >= a && slots[j] > v) { slots[j + 1] = slots[j]; --j; }
      slots[j + 1] = v;
    }
  }
}

// Small inputs (n <= kInvSmallN tokens, at most kInvSmallSlots slots): the whole inverse index in one CTA and one
// launch.  Counts and cursors live in shared memory; the order in which atomics hand out places does not
// matter because every token's list is sorted at the end.
constexpr int kInvSmallN = 4096, kInvSmallSlots = 1 << 14;
__global__ void __launch_bounds__(1024)
inv_small_kernel(const int32_t* __restrict__ I, int n, int total, int32_t* row_ptr, int32_t* slots, int* status) {
  extern __shared__ int s_cnt[];                       // [n] counts, then cursors
  __shared__ int s_warp[33];
  const int tid = threadIdx.x;
  for (int t = tid; t < n; t += 1024) s_cnt[t] = 0;
  __syncthreads();
  for (int s = tid; s < total; s += 1024) { const int t = I[s]; if (t >= 0 && idx_ok(t, 0, n, status)) atomicAdd(&s_cnt[t], 1); }
  __syncthreads();
  // exclusive scan over the tokens, 1024 * per at a time
  const int per = (n + 1023) / 1024, a = min(n, tid * per), b = min(n, a + per);
  int sum = 0;
  for (int t = a; t < b; ++t) sum += s_cnt[t];
  int total_sum;
  int run = block_exclusive_scan(sum, s_warp, total_sum);
  for (int t = a; t < b; ++t) { const int c = s_cnt[t]; row_ptr[t] = run; s_cnt[t] = run; run += c; }   // s_cnt becomes the cursor
  if (tid == 0) row_ptr[n] = total_sum;
  __syncthreads();
  for (int s = tid; s < total; s += 1024) { const int t = I[s]; if (t >= 0 && idx_ok(t, 0, n, nullptr)) slots[atomicAdd(&s_cnt[t], 1)] = s; }
  __syncthreads();
  __threadfence_block();
  for (int t = tid; t < n; t += 1024) {                // after the fill s_cnt[t] is the end of token t's list
    const int lo = t == 0 ? 0 : s_cnt[t - 1], hi = s_cnt[t];
    for (int i = lo + 1; i < hi; ++i) {
      const int v = slots[i]; int j = i - 1;
      while (j >= lo && slots[j] > v) { slots[j + 1] = slots[j]; --j; }
      slots[j + 1] = v;
    }
  }
}

// Medium inputs (n <= kInvClusterN): one cluster of eight CTAs runs the five steps in one launch, with hardware
// cluster barriers between them (counts and cursors in global memory, the eight tile sums of the scan read
// from the other CTAs' shared memory).
constexpr int kInvClusterN = 16384, kInvClusterSlots = 1 << 17, kInvClusterCtas = 8;
__device__ __forceinline__ void inv_cluster_sync() {
  asm volatile("barrier.cluster.arrive.release.aligned;\n barrier.cluster.wait.acquire.aligned;" ::: "memory");
}
__global__ void __launch_bounds__(1024)
inv_cluster_kernel(const int32_t* __restrict__ I, int n, int total, int32_t* row_ptr, int32_t* slots, int32_t* cnt, int* status) {
  __shared__ int s_warp[33];
  __shared__ int s_tile;                               // sum of this CTA's part of the counts
  const int tid = threadIdx.x, rank = blockIdx.x, nc = gridDim.x;      // the grid is the one cluster
  const int gtid = rank * 1024 + tid, gsize = nc * 1024;
  for (int t = gtid; t < n; t += gsize) cnt[t] = 0;
  inv_cluster_sync();
  for (int s = gtid; s < total; s += gsize) { const int t = I[s]; if (t >= 0 && idx_ok(t, 0, n, status)) atomicAdd(&cnt[t], 1); }
  inv_cluster_sync();
  // exclusive scan: CTA `rank` takes tokens [lo, hi), a thread `per` consecutive ones of them
  const int per_cta = (n + nc - 1) / nc, lo = min(n, rank * per_cta), hi = min(n, lo + per_cta);
  const int per = (per_cta + 1023) / 1024, a = min(hi, lo + tid * per), b = min(hi, a + per);
  int sum = 0;
  for (int t = a; t < b; ++t) sum += cnt[t];
  int tile;
  int run = block_exclusive_scan(sum, s_warp, tile);
  if (tid == 0) s_tile = tile;
  inv_cluster_sync();
  int before = 0;
  for (int r = 0; r < rank; ++r) {
    unsigned remote; int v;
    asm volatile("mapa.shared::cluster.u32 %0, %1, %2;" : "=r"(remote) : "r"((unsigned)__cvta_generic_to_shared(&s_tile)), "r"(r));
    asm volatile("ld.shared::cluster.s32 %0, [%1];" : "=r"(v) : "r"(remote));
    before += v;
  }
  run += before;
  for (int t = a; t < b; ++t) { const int c = cnt[t]; row_ptr[t] = run; cnt[t] = run; run += c; }      // cnt becomes the cursor
  if (rank == nc - 1 && tid == 0) row_ptr[n] = before + tile;
  inv_cluster_sync();
  for (int s = gtid; s < total; s += gsize) { const int t = I[s]; if (t >= 0 && idx_ok(t, 0, n, nullptr)) slots[atomicAdd(&cnt[t], 1)] = s; }
  inv_cluster_sync();
  for (int t = gtid; t < n; t += gsize) {
    const int p0 = row_ptr[t], p1 = row_ptr[t + 1];
    for (int i = p0 + 1; i < p1; ++i) {
      const int v = slots[i]; int j = i - 1;
      while (j >= p0 && slots[j] > v) { slots[j + 1] = slots[j]; --j; }
      slots[j + 1] = v;
    }
  }
}

cudaError_t launch_inverse_index(const int32_t* I, int64_t n, int64_t total, int32_t* row_ptr, int32_t* slots,
                                 void* scratch, int* status, cudaStream_t st) {
  if (n > kInvSmallN && n <= kInvClusterN && total <= kInvClusterSlots) {
    cudaLaunchConfig_t cfg; memset(&cfg, 0, sizeof(cfg));
    cfg.gridDim = dim3(kInvClusterCtas); cfg.blockDim = dim3(1024); cfg.stream = st;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeClusterDimension;
    attr[0].val.clusterDim.x = kInvClusterCtas; attr[0].val.clusterDim.y = 1; attr[0].val.clusterDim.z = 1;
    cfg.attrs = attr; cfg.numAttrs = 1;
    count_launch();
    return cudaLaunchKernelEx(&cfg, inv_cluster_kernel, I, (int)n, (int)total, row_ptr, slots, (int32_t*)scratch, status);
  }
  if (n <= kInvSmallN && total <= kInvSmallSlots) {
    const int smem = (int)n * 4;
    cudaError_t e0 = cudaFuncSetAttribute(inv_small_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, smem);
    if (e0 != cudaSuccess) return e0;
    count_launch();
    inv_small_kernel<<<1, 1024, smem, st>>>(I, (int)n, (int)total, row_ptr, slots, status);
    return cudaGetLastError();
  }
  int32_t* cnt = (int32_t*)scratch;
  int32_t* tile_sum = (int32_t*)((char*)scratch + inv_cnt_bytes(n));
  const unsigned tiles = (unsigned)((n + kScanTile - 1) / kScanTile);
  cudaError_t e;
  if ((e = cudaMemsetAsync(cnt, 0, (size_t)(n + 1) * 4, st)) != cudaSuccess) return e;
  count_launch();
  inv_count_kernel<<<grid_for(total, 256), 256, 0, st>>>(I, total, cnt, n, status);
  count_launch();
  inv_scan_tile_kernel<<<tiles, kScanThreads, 0, st>>>(cnt, n, row_ptr, tile_sum);
  count_launch();
  inv_scan_add_kernel<<<tiles, kScanThreads, 0, st>>>(tile_sum, n, row_ptr);
  count_launch();
  inv_fill_kernel<<<grid_for(total, 256), 256, 0, st>>>(I, total, row_ptr, cnt, slots, n);
  count_launch();
  inv_sort_kernel<<<grid_for(n, 256), 256, 0, st>>>(row_ptr, n, slots);
  return cudaGetLastError();
}

// ------------------------------------------------------------------------------------------
// Validation of an index structure (on request, and what the debug build's checks are modelled on): every access
// below is range-checked, so any contents are safe to hand in.  Violations are counted.
// ------------------------------------------------------------------------------------------
__global__ void validate_routing_kernel(const int32_t* __restrict__ I, const int32_t* __restrict__ row_ptr,
                                        const int32_t* __restrict__ slots, int64_t n, int64_t ng, int E, int64_t k_total,
                                        int64_t kg, int groups, int allow_empty, int* violations) {
  const int64_t total = (int64_t)E * k_total;
  const int64_t stride = (int64_t)gridDim.x * blockDim.x, g0 = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
  int bad = 0;
  // slots: a token of the slot's own routing group, or -1 where empty slots exist
  for (int64_t s = g0; s < total; s += stride) {
    const int t = I[s];
    const int64_t grp = (s % k_total) / kg;
    if (t == -1) { if (!allow_empty) ++bad; }
    else if (t < 0 || t >= n || t / ng != grp) ++bad;
  }
  // the token -> slot lists
  for (int64_t t = g0; t < n; t += stride) {
    const int64_t a = row_ptr[t], b = row_ptr[t + 1];
    if (t == 0 && a != 0) ++bad;
    if (a < 0 || b < a || b > total) { ++bad; continue; }
    int prev = -1;
    for (int64_t q = a; q < b; ++q) {
      const int s = slots[q];
      if (s < 0 || s >= total) { ++bad; continue; }
      if (s <= prev) ++bad;                             // ascending slot ids, hence ascending expert
      if (I[s] != t) ++bad;
      prev = s;
    }
  }
  if (bad) atomicAdd(violations, bad);
}

// every filled slot is listed exactly once: row_ptr[n] equals the number of filled slots
__global__ void validate_count_kernel(const int32_t* __restrict__ I, const int32_t* __restrict__ row_ptr, int64_t n, int64_t total,
                                      int* filled) {
  int c = 0;
  for (int64_t s = (int64_t)blockIdx.x * blockDim.x + threadIdx.x; s < total; s += (int64_t)gridDim.x * blockDim.x) c += I[s] >= 0;
  if (c) atomicAdd(filled, c);
}
__global__ void validate_total_kernel(const int32_t* __restrict__ row_ptr, int64_t n, const int* filled, int* violations) {
  if (row_ptr[n] != *filled) atomicAdd(violations, 1);
}

cudaError_t launch_validate_routing(const int32_t* I, const int32_t* row_ptr, const int32_t* slots, int64_t n, int64_t ng,
                                    int E, int64_t k_total, int64_t kg, int groups, int allow_empty, int* violations,
                                    cudaStream_t st) {
  const int64_t total = (int64_t)E * k_total;
  cudaError_t e = cudaMemsetAsync(violations, 0, 2 * sizeof(int), st);       // [0] violations, [1] filled slots
  if (e != cudaSuccess) return e;
  count_launch(3);
  validate_routing_kernel<<<grid_for(total > n ? total : n, 256), 256, 0, st>>>(I, row_ptr, slots, n, ng, E, k_total, kg, groups,
                                                                                 allow_empty, violations);
  validate_count_kernel<<<grid_for(total, 256), 256, 0, st>>>(I, row_ptr, n, total, violations + 1);
  validate_total_kernel<<<1, 1, 0, st>>>(row_ptr, n, violations + 1, violations);
  return cudaGetLastError();
}

// ------------------------------------------------------------------------------------------
// Shuffle, Eq. 3: X_in = P . X as an indexed row copy in 16-byte vectors.
// ------------------------------------------------------------------------------------------
__global__ void gather_kernel(const uint4* __restrict__ X, const int32_t* __restrict__ I, uint4* __restrict__ X_in,
                              int64_t total_vec, int vec_per_row, int64_t n, int* status) {
  for (int64_t g = (int64_t)blockIdx.x * blockDim.x + threadIdx.x; g < total_vec; g += (int64_t)gridDim.x * blockDim.x) {
    const int64_t s = g / vec_per_row; const int v = (int)(g % vec_per_row);
    int t = I[s];                                      // -1: an empty slot (token-choice routing only) holds a zero row
    if (t >= 0 && !idx_ok(t, 0, n, v == 0 ? status : nullptr)) t = -1;
    X_in[g] = t >= 0 ? X[(int64_t)t * vec_per_row + v] : make_uint4(0, 0, 0, 0);
  }
}

cudaError_t launch_gather(int dtype, const void* X, const int32_t* I, void* X_in, int64_t total, int d, int64_t n, int* status,
                          cudaStream_t st) {
  const int vpr = d * (dtype == 0 ? 4 : 2) / 16;
  const int64_t tv = total * vpr;
  count_launch();
  gather_kernel<<<grid_for(tv, 256, 148 * 32), 256, 0, st>>>((const uint4*)X, I, (uint4*)X_in, tv, vpr, n, status);
  return cudaGetLastError();
}

// ------------------------------------------------------------------------------------------
// Unshuffle, Eq. 4: X_out[t,:] = sum over the slots of t (ascending expert) of G[s] * X_e[s,:].
// Read through the token->slot index, so no atomics and a fixed summation order.
// ------------------------------------------------------------------------------------------
// four consecutive elements of a row of T
__device__ __forceinline__ void load4(const float* p, float* f) {
  const float4 v = *reinterpret_cast<const float4*>(p); f[0] = v.x; f[1] = v.y; f[2] = v.z; f[3] = v.w;
}
__device__ __forceinline__ void load4(const bf16* p, float* f) {
  const uint2 v = *reinterpret_cast<const uint2*>(p);
  f[0] = __uint_as_float(v.x << 16); f[1] = __uint_as_float(v.x & 0xFFFF0000u);
  f[2] = __uint_as_float(v.y << 16); f[3] = __uint_as_float(v.y & 0xFFFF0000u);
}
__device__ __forceinline__ void store4(float* p, const float* f) {
  *reinterpret_cast<float4*>(p) = make_float4(f[0], f[1], f[2], f[3]);
}
__device__ __forceinline__ void store4(bf16* p, const float* f) {
  __nv_bfloat162 a = __floats2bfloat162_rn(f[0], f[1]), b = __floats2bfloat162_rn(f[2], f[3]);
  *reinterpret_cast<uint2*>(p) = make_uint2(*reinterpret_cast<unsigned*>(&a), *reinterpret_cast<unsigned*>(&b));
}

template <typename T>
__global__ void combine_kernel(const float* __restrict__ X_e, const float* __restrict__ G,
                               const int32_t* __restrict__ row_ptr, const int32_t* __restrict__ slots,
                               T* __restrict__ X_out, int64_t total_quads, int quads_per_row, int64_t slots_total, int* status) {
  for (int64_t g = (int64_t)blockIdx.x * blockDim.x + threadIdx.x; g < total_quads; g += (int64_t)gridDim.x * blockDim.x) {
    const int64_t t = g / quads_per_row; const int v = (int)(g % quads_per_row);
    float acc[4] = {0.f, 0.f, 0.f, 0.f};
    int a = row_ptr[t], b = row_ptr[t + 1];
    if (!idx_ok(a, 0, slots_total + 1, v == 0 ? status : nullptr) || !idx_ok(b, a, slots_total + 1, v == 0 ? status : nullptr)) a = b = 0;
    // four slots at a time: their ids, then their weights and row pieces, are fetched together, and
    // added in slot order
    for (int q0 = a; q0 < b; q0 += 4) {
      int s[4]; float w[4]; float4 x[4];
#pragma unroll
      for (int u = 0; u < 4; ++u) {
        s[u] = q0 + u < b ? slots[q0 + u] : -1;
        if (s[u] >= 0 && !idx_ok(s[u], 0, slots_total, v == 0 ? status : nullptr)) s[u] = -1;
      }
#pragma unroll
      for (int u = 0; u < 4; ++u) {
        w[u] = s[u] >= 0 ? G[s[u]] : 0.f;
        x[u] = s[u] >= 0 ? *reinterpret_cast<const float4*>(X_e + ((int64_t)s[u] * quads_per_row + v) * 4) : make_float4(0.f, 0.f, 0.f, 0.f);
      }
#pragma unroll
      for (int u = 0; u < 4; ++u) {
        if (s[u] >= 0) {
          acc[0] = fmaf(w[u], x[u].x, acc[0]); acc[1] = fmaf(w[u], x[u].y, acc[1]);
          acc[2] = fmaf(w[u], x[u].z, acc[2]); acc[3] = fmaf(w[u], x[u].w, acc[3]);
        }
      }
    }
    store4(X_out + g * 4, acc);
  }
}

cudaError_t launch_combine(int dtype, const float* X_e, const float* G, const int32_t* row_ptr, const int32_t* slots,
                           void* X_out, int64_t n, int d, int64_t slots_total, int* status, cudaStream_t st) {
  const int qpr = d / 4;
  const int64_t tq = n * qpr;
  const unsigned grid = grid_for(tq, 256, 148 * 32);
  if (dtype == 0) { count_launch(); combine_kernel<float><<<grid, 256, 0, st>>>(X_e, G, row_ptr, slots, (float*)X_out, tq, qpr, slots_total, status); }
  else { count_launch(); combine_kernel<bf16><<<grid, 256, 0, st>>>(X_e, G, row_ptr, slots, (bf16*)X_out, tq, qpr, slots_total, status); }
  return cudaGetLastError();
}

// ------------------------------------------------------------------------------------------
// Backward of Eq. 4 per slot s = (i, j) holding token t:
//   dX_e[s,:] = G[s] * dX_out[t,:],   dG[s] = <dX_out[t,:], X_e[s,:]>.   One warp per slot.
// ------------------------------------------------------------------------------------------
template <typename T>
__global__ void bwd_combine_kernel(const T* __restrict__ dX_out, const float* __restrict__ X_e,
                                   const float* __restrict__ G, const int32_t* __restrict__ I,
                                   T* __restrict__ dX_e, float* __restrict__ dG, int64_t total, int quads_per_row, int64_t n,
                                   int* status) {
  const int lane = threadIdx.x & 31;
  const int64_t warps = ((int64_t)gridDim.x * blockDim.x) >> 5;
  for (int64_t s = ((int64_t)blockIdx.x * blockDim.x + threadIdx.x) >> 5; s < total; s += warps) {
    int64_t t = I[s];
    if (t >= 0 && !idx_ok(t, 0, n, lane == 0 ? status : nullptr)) t = -1;
    if (t < 0) {                                       // an empty slot (token-choice routing only): zero row, no gradient
      const float z[4] = {0.f, 0.f, 0.f, 0.f};
      for (int v = lane; v < quads_per_row; v += 32) store4(dX_e + (s * quads_per_row + v) * 4, z);
      if (lane == 0) dG[s] = 0.f;
      continue;
    }
    const float w = G[s];
    float dot = 0.f;
    for (int v = lane; v < quads_per_row; v += 32) {
      float dy[4], xe[4], o[4];
      load4(dX_out + (t * quads_per_row + v) * 4, dy);
      load4(X_e + (s * quads_per_row + v) * 4, xe);
#pragma unroll
      for (int i = 0; i < 4; ++i) { o[i] = w * dy[i]; dot = fmaf(dy[i], xe[i], dot); }
      store4(dX_e + (s * quads_per_row + v) * 4, o);
    }
    for (int o = 16; o; o >>= 1) dot += __shfl_xor_sync(0xffffffffu, dot, o);
    if (lane == 0) dG[s] = dot;
  }
}

cudaError_t launch_bwd_combine(int dtype, const void* dX_out, const float* X_e, const float* G, const int32_t* I,
                               void* dX_e, float* dG, int64_t total, int d, int64_t n, int* status, cudaStream_t st) {
  const int qpr = d / 4;
  const unsigned grid = grid_for(total * 32, 256, 148 * 16);
  if (dtype == 0) { count_launch(); bwd_combine_kernel<float><<<grid, 256, 0, st>>>((const float*)dX_out, X_e, G, I, (float*)dX_e, dG, total, qpr, n, status); }
  else { count_launch(); bwd_combine_kernel<bf16><<<grid, 256, 0, st>>>((const bf16*)dX_out, X_e, G, I, (bf16*)dX_e, dG, total, qpr, n, status); }
  return cudaGetLastError();
}

// ------------------------------------------------------------------------------------------
// Backward of the softmax of Eq. 2, one warp per token.  dS[t,i] is dG of the slot of expert i that
// holds t (0 if none);  dL[t,i] = S[t,i] * (dS[t,i] - sum_i' dS[t,i'] * S[t,i']).
// ------------------------------------------------------------------------------------------
__device__ __forceinline__ void st_dl(float* p, int64_t i, float v) { p[i] = v; }
__device__ __forceinline__ void st_dl(bf16* p, int64_t i, float v) { p[i] = __float2bfloat16(v); }

template <typename TL>
__global__ void bwd_softmax_kernel(const float* __restrict__ S, const float* __restrict__ dG,
                                   const int32_t* __restrict__ row_ptr, const int32_t* __restrict__ slots,
                                   TL* __restrict__ dL, int64_t n, int E, int64_t k, int* status) {
  const int lane = threadIdx.x & 31;
  const int64_t warps = ((int64_t)gridDim.x * blockDim.x) >> 5;
  const int64_t slots_total = (int64_t)E * k;
  for (int64_t t = ((int64_t)blockIdx.x * blockDim.x + threadIdx.x) >> 5; t < n; t += warps) {
    int a = row_ptr[t], b = row_ptr[t + 1];
    if (!idx_ok(a, 0, slots_total + 1, lane == 0 ? status : nullptr) || !idx_ok(b, a, slots_total + 1, lane == 0 ? status : nullptr)) a = b = 0;
    float dot = 0.f;
    for (int q = a + lane; q < b; q += 32) {
      const int s = slots[q];
      if (!idx_ok(s, 0, slots_total, status)) continue;
      dot = fmaf(dG[s], S[t * E + s / k], dot);
    }
    for (int o = 16; o; o >>= 1) dot += __shfl_xor_sync(0xffffffffu, dot, o);
    for (int i = lane; i < E; i += 32) st_dl(dL, t * E + i, -S[t * E + i] * dot);
    __syncwarp();
    for (int q = a + lane; q < b; q += 32) {           // the slots of one token belong to distinct experts
      const int s = slots[q]; const int64_t i = s / k;
      if (!idx_ok(s, 0, slots_total, nullptr)) continue;
      st_dl(dL, t * E + i, S[t * E + i] * (dG[s] - dot));
    }
  }
}

cudaError_t launch_bwd_softmax(const float* S, const float* dG, const int32_t* row_ptr, const int32_t* slots,
                               void* dL, int dl_bf16, int64_t n, int E, int64_t k, int* status, cudaStream_t st) {
  count_launch();
  const unsigned grid = grid_for(n * 32, 256, 148 * 16);
  if (dl_bf16) bwd_softmax_kernel<bf16><<<grid, 256, 0, st>>>(S, dG, row_ptr, slots, (bf16*)dL, n, E, k, status);
  else bwd_softmax_kernel<float><<<grid, 256, 0, st>>>(S, dG, row_ptr, slots, (float*)dL, n, E, k, status);
  return cudaGetLastError();
}

// ------------------------------------------------------------------------------------------
// Column sums per expert (gradients of the bias terms Eq. 3 leaves out): a thread owns a column and adds its rows in
// order, so the result does not depend on scheduling; neighbouring threads read neighbouring columns.
// ------------------------------------------------------------------------------------------
template <typename T>
__global__ void __launch_bounds__(256) column_sums_kernel(const T* __restrict__ A, T* __restrict__ out, int64_t rows, int cols,
                                                          const int32_t* __restrict__ batch_rows) {
  const int b = blockIdx.y, c = blockIdx.x * 256 + threadIdx.x;
  if (c >= cols) return;
  int64_t lim = rows;
  if (batch_rows != nullptr && batch_rows[b] < lim) lim = batch_rows[b];
  const T* p = A + (int64_t)b * rows * cols + c;
  float acc = 0.f;
  int64_t r = 0;
  for (; r + 8 <= lim; r += 8) {
    float v[8];
#pragma unroll
    for (int u = 0; u < 8; ++u) v[u] = ld_f(p, (r + u) * cols);
#pragma unroll
    for (int u = 0; u < 8; ++u) acc += v[u];
  }
  for (; r < lim; ++r) acc += ld_f(p, r * cols);
  if constexpr (sizeof(T) == 4) out[(int64_t)b * cols + c] = acc; else out[(int64_t)b * cols + c] = __float2bfloat16(acc);
}

cudaError_t launch_column_sums(int dtype, const void* A, void* out, int batches, int64_t rows, int cols,
                               const int32_t* batch_rows, cudaStream_t st) {
  const dim3 grid((cols + 255) / 256, batches);
  count_launch();
  if (dtype == 0) column_sums_kernel<float><<<grid, 256, 0, st>>>((const float*)A, (float*)out, rows, cols, batch_rows);
  else column_sums_kernel<bf16><<<grid, 256, 0, st>>>((const bf16*)A, (bf16*)out, rows, cols, batch_rows);
  return cudaGetLastError();
}

// ------------------------------------------------------------------------------------------
// Fixed-order sum of split partial results.
// ------------------------------------------------------------------------------------------
template <typename T>
__global__ void reduce_partials_kernel(const float* __restrict__ part, T* __restrict__ out, int P, int64_t elems) {
  for (int64_t g = (int64_t)blockIdx.x * blockDim.x + threadIdx.x; g < elems; g += (int64_t)gridDim.x * blockDim.x) {
    float acc = 0.f;
    for (int p = 0; p < P; ++p) acc += part[(int64_t)p * elems + g];
    if constexpr (sizeof(T) == 4) out[g] = acc; else out[g] = __float2bfloat16(acc);
  }
}

cudaError_t launch_reduce_partials(int dtype, const float* part, void* out, int P, int64_t elems, cudaStream_t st) {
  if (dtype == 0) { count_launch(); reduce_partials_kernel<float><<<grid_for(elems, 256), 256, 0, st>>>(part, (float*)out, P, elems); }
  else { count_launch(); reduce_partials_kernel<bf16><<<grid_for(elems, 256), 256, 0, st>>>(part, (bf16*)out, P, elems); }
  return cudaGetLastError();
}

}  // namespace ecmoe
