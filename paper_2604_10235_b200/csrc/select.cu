// A4: selection of the retained tokens of every (sequence, KV head) under the budget.
//
// Items (tokens, or fixed chunks of tokens) are ranked: protected first (in sequence order),
// then larger fused value, then lower index.  One CTA of 1024 threads owns one (sequence,
// head).  Every thread owns a contiguous range of items, so duplicates produced by max
// pooling (runs of equal neighbours) meet inside one thread rather than across a warp.
// The cut-off is found by a 4 x 8-bit radix descent over order-preserving integer keys
// that are first shifted to the range actually present (min..max), which spreads softmax
// scores - whose exponents are nearly all equal - over all 256 bins.  Histograms carry token
// counts, so chunks of unequal length (the ragged last chunk) need no special case.  The
// final ordered pass resolves ties towards lower indices with one block-wide prefix sum and
// writes ascending token indices.
#include "cc_internal.cuh"
#include "select_common.cuh"

namespace cc {

namespace {

constexpr int kThreads = 1024;
constexpr int kWarps = kThreads / 32;
constexpr int kHistCopies = 8;
constexpr int kHistStride = 257;

struct Shared {
  unsigned hist[kHistCopies * kHistStride];
  unsigned tot[256];
  unsigned warp_a[kWarps];
  unsigned warp_b[kWarps];
  unsigned bcast[4];
};



__device__ unsigned block_sum(Shared& sm, unsigned v) {
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  v = warp_sum(v);
  __syncthreads();
  if (lane == 0) sm.warp_a[warp] = v;
  __syncthreads();
  unsigned t = sm.warp_a[lane];
  t = warp_sum(t);
  return t;
}

__device__ void block_minmax(Shared& sm, unsigned& lo, unsigned& hi) {
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) {
    lo = min(lo, __shfl_xor_sync(0xffffffffu, lo, o));
    hi = max(hi, __shfl_xor_sync(0xffffffffu, hi, o));
  }
  __syncthreads();
  if (lane == 0) { sm.warp_a[warp] = lo; sm.warp_b[warp] = hi; }
  __syncthreads();
  lo = sm.warp_a[lane];
  hi = sm.warp_b[lane];
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) {
    lo = min(lo, __shfl_xor_sync(0xffffffffu, lo, o));
    hi = max(hi, __shfl_xor_sync(0xffffffffu, hi, o));
  }
}

// exclusive prefix sums over the threads of the block, for two counters at once
__device__ void block_scan2(Shared& sm, unsigned a, unsigned b, unsigned& ea, unsigned& eb) {
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  unsigned ia = a, ib = b;
#pragma unroll
  for (int o = 1; o < 32; o <<= 1) {
    unsigned ta = __shfl_up_sync(0xffffffffu, ia, o);
    unsigned tb = __shfl_up_sync(0xffffffffu, ib, o);
    if (lane >= o) { ia += ta; ib += tb; }
  }
  __syncthreads();
  if (lane == 31) { sm.warp_a[warp] = ia; sm.warp_b[warp] = ib; }
  __syncthreads();
  unsigned wa = sm.warp_a[lane], wb = sm.warp_b[lane];
  unsigned xa = wa, xb = wb;
#pragma unroll
  for (int o = 1; o < 32; o <<= 1) {
    unsigned ta = __shfl_up_sync(0xffffffffu, xa, o);
    unsigned tb = __shfl_up_sync(0xffffffffu, xb, o);
    if (lane >= o) { xa += ta; xb += tb; }
  }
  const unsigned base_a = __shfl_sync(0xffffffffu, xa - wa, warp);
  const unsigned base_b = __shfl_sync(0xffffffffu, xb - wb, warp);
  ea = base_a + ia - a;
  eb = base_b + ib - b;
}

// Finds the key T (and the token weight above it) such that
//   weight(key > T) < R <= weight(key >= T)      over the eligible items,
// where get(i, key, len) returns whether item i is eligible.  Requires 1 <= R <= total weight.
template <class Get>
__device__ void radix_threshold(Shared& sm, int lo, int hi, unsigned R, Get get,
                                unsigned& T, unsigned& w_above) {
  unsigned kmin = 0xffffffffu, kmax = 0u;
  for (int i = lo; i < hi; ++i) {
    unsigned key, len;
    if (get(i, key, len)) { kmin = min(kmin, key); kmax = max(kmax, key); }
  }
  block_minmax(sm, kmin, kmax);
  const unsigned range = kmax - kmin;
  const int sh = range ? __clz(range) : 0;
  unsigned prefix = 0;             // resolved high bits of the shifted key
  unsigned remaining = R;
  const int copy = (threadIdx.x >> 5) % kHistCopies;
  for (int pass = 3; pass >= 0 && range; --pass) {
    for (int b = threadIdx.x; b < kHistCopies * kHistStride; b += kThreads) sm.hist[b] = 0;
    __syncthreads();
    const int shift = pass * 8;
    for (int i = lo; i < hi; ++i) {
      unsigned key, len;
      if (!get(i, key, len)) continue;
      const unsigned kk = (key - kmin) << sh;
      const bool match = pass == 3 || (kk >> (shift + 8)) == (prefix >> (shift + 8));
      if (match) atomicAdd(&sm.hist[copy * kHistStride + ((kk >> shift) & 255u)], len);
    }
    __syncthreads();
    // thread t (< 256) takes bin 255 - t so that a forward scan walks keys downwards
    unsigned v = 0;
    if (threadIdx.x < 256) {
      const int bin = 255 - threadIdx.x;
#pragma unroll
      for (int c = 0; c < kHistCopies; ++c) v += sm.hist[c * kHistStride + bin];
    }
    unsigned excl, dummy;
    block_scan2(sm, v, 0u, excl, dummy);
    if (threadIdx.x < 256 && excl < remaining && remaining <= excl + v) {
      sm.bcast[0] = 255 - threadIdx.x;
      sm.bcast[1] = remaining - excl;
    }
    __syncthreads();
    prefix |= sm.bcast[0] << shift;
    remaining = sm.bcast[1];
    __syncthreads();
  }
  T = kmin + (prefix >> sh);
  w_above = R - remaining;
}

// grid: (H_kv, num_seqs); flags: one byte per (head, item) in the workspace
__global__ void __launch_bounds__(kThreads, 1)
select_kernel(const __grid_constant__ BatchTable bt, int hkv, float theta,
              const float* __restrict__ fused, const float* __restrict__ prior,
              int32_t* __restrict__ idx, int32_t* __restrict__ count,
              uint8_t* __restrict__ flags) {
  __shared__ Shared sm;
  const int h = blockIdx.x, s = blockIdx.y;
  const SeqInfo& q = bt.seq[s];
  const int m = q.n_items, cs = bt.chunk;
  const float* f = fused + (int64_t)h * bt.m_tot + q.item_off;
  const float* p = prior + q.tok_off;
  uint8_t* fl = flags + (int64_t)h * bt.m_tot + q.item_off;
  int32_t* out = idx + (int64_t)h * bt.b_tot + q.idx_off;
  const unsigned keep = (unsigned)q.keep;

  const int per = (m + kThreads - 1) / kThreads;
  const int lo = min(m, (int)threadIdx.x * per);
  const int hi = min(m, lo + per);

  auto item_len = [&](int i) -> unsigned { return (unsigned)(min(q.n, (i + 1) * cs) - i * cs); };
  auto item_prior = [&](int i) -> float {
    float pr = p[(int64_t)i * cs];
    const int end = min(q.n, (i + 1) * cs);
    for (int j = i * cs + 1; j < end; ++j) pr = fmaxf(pr, p[j]);
    return pr;
  };

  // ---- stage 0: protected items
  unsigned wf = 0;
  for (int i = lo; i < hi; ++i) {
    const bool fo = item_prior(i) >= theta;
    fl[i] = fo ? 1 : 0;
    if (fo) wf += item_len(i);
  }
  unsigned forced_tokens = block_sum(sm, wf);

  // ---- stage 1: cap on protected items (longest prefix by (prior desc, index asc) within B_span)
  if (q.span_cap >= 0 && forced_tokens > (unsigned)q.span_cap) {
    const unsigned cap = (unsigned)q.span_cap;
    unsigned t1, above1;
    radix_threshold(sm, lo, hi, cap + 1u,
                    [&](int i, unsigned& key, unsigned& len) {
                      if (!fl[i]) return false;
                      key = mono_key(item_prior(i));
                      len = item_len(i);
                      return true;
                    }, t1, above1);
    unsigned tie_w = 0;
    for (int i = lo; i < hi; ++i)
      if (fl[i] && mono_key(item_prior(i)) == t1) tie_w += item_len(i);
    unsigned tie_before, dummy;
    block_scan2(sm, tie_w, 0u, tie_before, dummy);
    unsigned kept = 0;
    for (int i = lo; i < hi; ++i) {
      if (!fl[i]) continue;
      const unsigned key = mono_key(item_prior(i));
      const unsigned len = item_len(i);
      if (key > t1) { kept += len; continue; }
      if (key == t1) {
        const bool fits = above1 + tie_before + len <= cap;
        tie_before += len;
        if (fits) { kept += len; continue; }
      }
      fl[i] = 0;
    }
    forced_tokens = block_sum(sm, kept);
  }

  // ---- stage 2: cut-off among the unprotected items
  bool ties_are_forced;
  unsigned t = 0, tie_budget;
  if (forced_tokens >= keep) {
    ties_are_forced = true;          // protected items alone fill the budget: first B in order
    tie_budget = keep;
  } else {
    ties_are_forced = false;
    unsigned above;
    radix_threshold(sm, lo, hi, keep - forced_tokens,
                    [&](int i, unsigned& key, unsigned& len) {
                      if (fl[i]) return false;
                      key = mono_key(f[i]);
                      len = item_len(i);
                      return true;
                    }, t, above);
    tie_budget = keep - forced_tokens - above;
  }

  // ---- stage 3: ordered emission
  unsigned def_w = 0, tie_w = 0;
  for (int i = lo; i < hi; ++i) {
    const unsigned len = item_len(i);
    if (fl[i]) {
      if (ties_are_forced) tie_w += len; else def_w += len;
    } else if (!ties_are_forced) {
      const unsigned key = mono_key(f[i]);
      if (key > t) def_w += len; else if (key == t) tie_w += len;
    }
  }
  unsigned def_before, tie_before;
  block_scan2(sm, def_w, tie_w, def_before, tie_before);
  for (int i = lo; i < hi; ++i) {
    const unsigned len = item_len(i);
    unsigned take = 0;
    bool tie = false;
    if (fl[i]) {
      if (ties_are_forced) tie = true; else take = len;
    } else if (!ties_are_forced) {
      const unsigned key = mono_key(f[i]);
      if (key > t) take = len; else if (key == t) tie = true;
    }
    const unsigned pos = def_before + min(tie_before, tie_budget);
    if (tie) {
      take = tie_before < tie_budget ? min(len, tie_budget - tie_before) : 0u;
      tie_before += len;
    } else {
      def_before += take;
    }
    for (unsigned k = 0; k < take; ++k)
      if (pos + k < keep) out[pos + k] = i * cs + (int)k;
  }
  for (int i = (int)keep + threadIdx.x; i < q.budget; i += kThreads) out[i] = -1;
  if (threadIdx.x == 0) count[s * hkv + h] = (int)keep;
}

// Scratch for cc_topk_select_static: one flag byte per (head, item), resident in every GPU
// that loads the library until the process exits.  Shared by all calls; the kernel writes
// each flag before it reads it, so stale contents of an earlier call do no harm.
static __device__ __align__(256) uint8_t g_static_select_flags[CC_STATIC_SELECT_MAX_ITEMS];

}  // namespace

int64_t select_static_capacity() { return (int64_t)CC_STATIC_SELECT_MAX_ITEMS; }

cudaError_t launch_select_static(const Launch& L, const BatchTable& bt, const Geometry& g,
                                 float force_threshold, const float* fused, const float* prior,
                                 int32_t* idx, int32_t* count, int device) {
  // In host code the array's name is only a handle; its device address is looked up once per
  // device (with that device current) and cached.
  // The launch goes to the current device, so that has to be the context's device on every
  // call, not only on the one that resolves the address.
  static uint8_t* cached[64] = {nullptr};
  if (device < 0 || device >= 64) return cudaErrorInvalidDevice;
  int cur = -1;
  cudaError_t e = cudaGetDevice(&cur);
  if (e != cudaSuccess) return e;
  if (cur != device) return cudaErrorInvalidDevice;
  uint8_t* ptr = cached[device];
  if (ptr == nullptr) {
    e = cudaGetSymbolAddress((void**)&ptr, g_static_select_flags);
    if (e != cudaSuccess) return e;
    if (ptr == nullptr) return cudaErrorInvalidSymbol;
    cached[device] = ptr;
  }
  dim3 grid(g.hkv, bt.num_seqs);
  select_kernel<<<grid, kThreads, 0, L.stream>>>(bt, g.hkv, force_threshold, fused, prior, idx,
                                                 count, ptr);
  return cudaGetLastError();
}

size_t select_ws_bytes(const BatchTable& bt, const Geometry& g) {
  return (((size_t)g.hkv * (size_t)bt.m_tot) + 255) / 256 * 256;
}

cudaError_t launch_select(const Launch& L, const BatchTable& bt, const Geometry& g,
                          float force_threshold, const float* fused, const float* prior,
                          int32_t* idx, int32_t* count, void* ws) {
  dim3 grid(g.hkv, bt.num_seqs);
  select_kernel<<<grid, kThreads, 0, L.stream>>>(bt, g.hkv, force_threshold, fused, prior, idx,
                                                 count, (uint8_t*)ws);
  return cudaGetLastError();
}

}  // namespace cc
