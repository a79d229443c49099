// A2 + A3 + A4 on a thread-block cluster: pooling, prior fusion and selection of the retained
// tokens of one (sequence, KV head) by up to eight CTAs that keep their slice of the items in
// shared memory.
//
// Ranking (protected first in sequence order, then larger fused value, then lower index) and the
// output (ascending token indices) are those of select.cu; what differs is where the data
// lives and how the CTAs cooperate:
//   * every item is read from global memory once; its order-preserving integer key and its
//     protected flag stay in shared memory, so the radix descent and the ordered emission never
//     go back to L2;
//   * cluster-wide sums, min/max and histograms are exchanged through distributed shared
//     memory: a CTA publishes into its own buffer, one cluster barrier later every CTA reads all
//     peers.  Buffers alternate between two copies, which makes one barrier per exchange enough;
//   * the cut-off is found by an four-step 8-bit radix descent over keys shifted to the range that
//     is present, and stops early once a bin has to be taken whole;
//   * with FUSED the kernel starts from the raw scores: it pools them (max / avg, or sums them
//     over a chunk), fuses them with the prior using the same explicitly rounded f32 operations
//     as fuse_pool.cu, and also stores the fused values.
#include <cooperative_groups.h>
#include <string.h>

#include "cc_internal.cuh"
#include "select_common.cuh"

namespace cg = cooperative_groups;

namespace cc {

namespace {

constexpr int kThreads = 1024;
constexpr int kWarps = kThreads / 32;
constexpr int kDigitBits = 8;
constexpr int kBins = 1 << kDigitBits;
constexpr int kCopies = 2;
constexpr int kMaxCluster = 8;
constexpr int kCtaItems = 32768;          // items one CTA keeps in shared memory
constexpr int kStagedItems = 16384;       // up to here the raw scores of the slice are staged there too

struct Shared {
  unsigned hist[2][kCopies][kBins];
  unsigned xchg[2][kMaxCluster][4];   // [buffer copy][source CTA][word]: written by the peers
  unsigned warp_a[kWarps];
  unsigned warp_b[kWarps];
  unsigned bcast[4];
};

struct ClusterParams {
  int cluster;               // CTAs per (sequence, head)
  int hkv;
  float theta;
  // FUSED only
  int stage_u;               // the slice's raw scores are staged in shared memory before pooling
  int pool_kind, pool_size;
  float alpha, beta;
  const float* scores;
  float* fused_out;
  // plain
  const float* fused_in;
  const float* prior;
  int32_t* idx;
  int32_t* count;
};

__host__ __device__ __forceinline__ int padded(int li) { return li + (li >> 5); }


struct Ctx {
  Shared* sm;
  int C, rank;
  unsigned phase;          // number of exchanges done so far (selects the buffer copy)

  __device__ void sync_all() {
    if (C > 1) cg::this_cluster().sync(); else __syncthreads();
  }
  __device__ unsigned peer(const unsigned* p, int r) const {
    if (C == 1) return *p;
    return *cg::this_cluster().map_shared_rank(const_cast<unsigned*>(p), r);
  }

  // Exchange of up to three words per CTA: threads 0..C-1 each store this CTA's words into one
  // peer's shared memory (remote stores need no round trip), the cluster barrier publishes them,
  // and every thread then reads all CTAs' words locally.  Two buffer copies: a CTA writes copy
  // k & 1 for exchange k only after the barrier of exchange k - 1, which every peer reaches
  // after it has read exchange k - 2.
  __device__ unsigned publish(unsigned w0, unsigned w1, unsigned w2) {
    const unsigned bf = phase++ & 1u;
    if ((int)threadIdx.x < C) {
      unsigned* dst = cg::this_cluster().map_shared_rank(&sm->xchg[bf][rank][0], (int)threadIdx.x);
      dst[0] = w0;
      dst[1] = w1;
      dst[2] = w2;
    }
    sync_all();
    return bf;
  }

  // sum over the block; every thread gets the result
  __device__ unsigned block_sum(unsigned v) {
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    v = warp_sum(v);
    __syncthreads();
    if (lane == 0) sm->warp_a[warp] = v;
    __syncthreads();
    return warp_sum(sm->warp_a[lane]);
  }
  // sum over all threads of the cluster
  __device__ unsigned cluster_sum(unsigned v) {
    v = block_sum(v);
    if (C == 1) return v;
    const unsigned b = publish(v, 0u, 0u);
    unsigned t = 0;
#pragma unroll
    for (int r = 0; r < kMaxCluster; ++r)
      if (r < C) t += sm->xchg[b][r][0];
    return t;
  }
  __device__ void cluster_minmax(unsigned& lo, unsigned& hi) {
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) {
      lo = min(lo, __shfl_xor_sync(0xffffffffu, lo, o));
      hi = max(hi, __shfl_xor_sync(0xffffffffu, hi, o));
    }
    __syncthreads();
    if (lane == 0) { sm->warp_a[warp] = lo; sm->warp_b[warp] = hi; }
    __syncthreads();
    lo = sm->warp_a[lane];
    hi = sm->warp_b[lane];
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) {
      lo = min(lo, __shfl_xor_sync(0xffffffffu, lo, o));
      hi = max(hi, __shfl_xor_sync(0xffffffffu, hi, o));
    }
    if (C == 1) return;
    const unsigned b = publish(lo, hi, 0u);
#pragma unroll
    for (int r = 0; r < kMaxCluster; ++r) {
      if (r < C) {
        lo = min(lo, sm->xchg[b][r][0]);
        hi = max(hi, sm->xchg[b][r][1]);
      }
    }
  }
  // exclusive prefix sums over the threads of the block for two counters; tot_* = block totals
  __device__ void block_scan2(unsigned a, unsigned b, unsigned& ea, unsigned& eb,
                              unsigned& tot_a, unsigned& tot_b) {
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    unsigned ia = a, ib = b;
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) {
      unsigned ta = __shfl_up_sync(0xffffffffu, ia, o);
      unsigned tb = __shfl_up_sync(0xffffffffu, ib, o);
      if (lane >= o) { ia += ta; ib += tb; }
    }
    __syncthreads();
    if (lane == 31) { sm->warp_a[warp] = ia; sm->warp_b[warp] = ib; }
    __syncthreads();
    const unsigned wa = sm->warp_a[lane], wb = sm->warp_b[lane];
    unsigned xa = wa, xb = wb;
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) {
      unsigned ta = __shfl_up_sync(0xffffffffu, xa, o);
      unsigned tb = __shfl_up_sync(0xffffffffu, xb, o);
      if (lane >= o) { xa += ta; xb += tb; }
    }
    tot_a = __shfl_sync(0xffffffffu, xa, 31);
    tot_b = __shfl_sync(0xffffffffu, xb, 31);
    ea = __shfl_sync(0xffffffffu, xa - wa, warp) + ia - a;
    eb = __shfl_sync(0xffffffffu, xb - wb, warp) + ib - b;
  }
  // exclusive prefix of one counter over all threads of the cluster, and its cluster total
  // and, in the same exchange, the cluster-wide minimum of lo and maximum of hi (carried through
  // the block scan as its second counter's inputs would not do: they are reduced separately)
  __device__ void cluster_scan_total(unsigned a, unsigned& ea, unsigned& total, unsigned& lo,
                                     unsigned& hi) {
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) {
      lo = min(lo, __shfl_xor_sync(0xffffffffu, lo, o));
      hi = max(hi, __shfl_xor_sync(0xffffffffu, hi, o));
    }
    __shared__ unsigned w_lo[kWarps], w_hi[kWarps];
    if (lane == 0) { w_lo[warp] = lo; w_hi[warp] = hi; }
    unsigned eb, ta, tb;
    block_scan2(a, 0u, ea, eb, ta, tb);      // its barriers also publish w_lo / w_hi
    lo = w_lo[lane];
    hi = w_hi[lane];
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) {
      lo = min(lo, __shfl_xor_sync(0xffffffffu, lo, o));
      hi = max(hi, __shfl_xor_sync(0xffffffffu, hi, o));
    }
    total = ta;
    if (C == 1) return;
    const unsigned bf = publish(ta, lo, hi);
    total = 0;
#pragma unroll
    for (int r = 0; r < kMaxCluster; ++r) {
      if (r < C) {
        const unsigned v = sm->xchg[bf][r][0];
        total += v;
        if (r < rank) ea += v;
        lo = min(lo, sm->xchg[bf][r][1]);
        hi = max(hi, sm->xchg[bf][r][2]);
      }
    }
  }
  // the same over all threads of the cluster (CTA rank major)
  __device__ void cluster_scan2(unsigned a, unsigned b, unsigned& ea, unsigned& eb) {
    unsigned ta, tb;
    block_scan2(a, b, ea, eb, ta, tb);
    if (C == 1) return;
    const unsigned bf = publish(ta, tb, 0u);
#pragma unroll
    for (int r = 0; r < kMaxCluster - 1; ++r) {
      if (r < rank) {
        ea += sm->xchg[bf][r][0];
        eb += sm->xchg[bf][r][1];
      }
    }
  }
};

// Finds T over the eligible items such that weight(key > T) < R <= weight(key >= T), with
// 1 <= R <= total eligible weight.  get(li, key, len) tells whether local item li is
// eligible.  When `whole_bin` comes back true the descent stopped early: every eligible item
// with key >= T is taken and nothing is tied.  w_above = weight strictly above the ties.
template <class Get>
__device__ void radix_threshold(Ctx& c, int lo, int hi, unsigned R, bool allow_early, Get get,
                                unsigned& T, unsigned& w_above, bool& whole_bin,
                                bool range_known = false, unsigned kmin = 0xffffffffu,
                                unsigned kmax = 0u) {
  Shared& sm = *c.sm;
  if (!range_known) {
    for (int li = lo; li < hi; ++li) {
      unsigned key, len;
      if (get(li, key, len)) { kmin = min(kmin, key); kmax = max(kmax, key); }
    }
    c.cluster_minmax(kmin, kmax);
  }
  const unsigned range = kmax - kmin;
  const int sh = range ? __clz(range) : 0;
  unsigned prefix = 0, remaining = R;
  whole_bin = false;
  const int copy = (threadIdx.x >> 5) & (kCopies - 1);
  int shift = 32;
#pragma unroll 1
  while (shift > 0 && range) {
    const int bits = min(kDigitBits, shift);
    const int hi_shift = shift;             // bits [31, hi_shift) are resolved
    shift -= bits;
    const unsigned b = c.phase++ & 1u;
    unsigned* h = &sm.hist[b][0][0];
#pragma unroll 1
    for (int i = threadIdx.x; i < kCopies * kBins; i += kThreads) h[i] = 0;
    __syncthreads();
    for (int li = lo; li < hi; ++li) {
      unsigned key, len;
      if (!get(li, key, len)) continue;
      const unsigned kk = (key - kmin) << sh;
      const bool match = hi_shift == 32 || (kk >> hi_shift) == (prefix >> hi_shift);
      if (match) atomicAdd(&sm.hist[b][copy][(kk >> shift) & ((1u << bits) - 1u)], len);
    }
    // fold the private copies into copy 0 before the peers look at it
    __syncthreads();
    if (threadIdx.x < kBins) {
      unsigned t = sm.hist[b][0][threadIdx.x];
#pragma unroll
      for (int cp = 1; cp < kCopies; ++cp) t += sm.hist[b][cp][threadIdx.x];
      sm.hist[b][0][threadIdx.x] = t;
    }
    c.sync_all();
    // thread t (< 256) owns bin 255 - t, so a forward scan walks the keys downwards
    const int bin0 = kBins - 1 - (int)threadIdx.x;
    unsigned v0 = 0;
    if (threadIdx.x < kBins)
#pragma unroll
      for (int r = 0; r < kMaxCluster; ++r)
        if (r < c.C) v0 += c.peer(&sm.hist[b][0][bin0], r);
    unsigned excl, d0, d1, d2;
    c.block_scan2(v0, 0u, excl, d0, d1, d2);
    if (threadIdx.x < kBins && excl < remaining && remaining <= excl + v0) {
      sm.bcast[0] = (unsigned)bin0; sm.bcast[1] = remaining - excl; sm.bcast[2] = v0;
    }
    __syncthreads();
    prefix |= sm.bcast[0] << shift;
    remaining = sm.bcast[1];
    const unsigned in_bin = sm.bcast[2];
    __syncthreads();
    if (allow_early && remaining == in_bin && shift > 0) {
      whole_bin = true;
      remaining = 0;
      break;
    }
  }
  T = kmin + (prefix >> sh);
  w_above = R - remaining;
  if (whole_bin) w_above = R;
}

// CHUNKED instantiations rank fixed chunks of bt.chunk tokens; the others are compiled for
// token-level items only (bt.chunk == 1), which keeps their code short.
template <bool FUSED, bool CHUNKED>
__global__ void __launch_bounds__(kThreads, 1)
select_cluster_kernel(const __grid_constant__ BatchTable bt, const __grid_constant__ ClusterParams P) {
  extern __shared__ __align__(16) uint8_t dyn[];
  Shared* smp = reinterpret_cast<Shared*>(dyn);
  unsigned* keys = reinterpret_cast<unsigned*>(dyn + sizeof(Shared));
  Ctx c;
  c.sm = smp;
  c.C = P.cluster;
  c.rank = P.cluster > 1 ? (int)cg::this_cluster().block_rank() : 0;
  c.phase = 0;

  pdl_launch_dependents();
  // FUSED runs right after the second score pass, which starts only once the caller's inputs
  // are complete: the token-level path reads the prior before it waits for the scores
  const bool early_prior = FUSED && !CHUNKED;
  if (!early_prior) pdl_wait();

  const int h = blockIdx.y, s = blockIdx.z;
  const SeqInfo& q = bt.seq[s];
  const int m = q.n_items, cs = CHUNKED ? bt.chunk : 1;
  const int per = (m + c.C * kThreads - 1) / (c.C * kThreads);       // items per thread
  const int cta_lo = min(m, c.rank * kThreads * per);
  const int cta_hi = min(m, cta_lo + kThreads * per);
  const int cta_items = cta_hi - cta_lo;
  uint8_t* flags = reinterpret_cast<uint8_t*>(keys + padded(kThreads * per) + 1);
  const float* p = P.prior + q.tok_off;
  int32_t* out = P.idx + (int64_t)h * bt.b_tot + q.idx_off;
  const unsigned keep = (unsigned)q.keep;
  const float theta = P.theta;

  // contiguous local range of this thread
  const int lo = min(cta_items, (int)threadIdx.x * per);
  const int hi = min(cta_items, lo + per);

  auto item_len = [&](int li) -> unsigned {
    if (cs == 1) return 1u;
    const int i = cta_lo + li;
    return (unsigned)(min(q.n, (i + 1) * cs) - i * cs);
  };
  auto item_prior = [&](int li) -> float {
    const int i = cta_lo + li;
    if (cs == 1) return p[i];
    float pr = p[(int64_t)i * cs];
    const int end = min(q.n, (i + 1) * cs);
    for (int j = i * cs + 1; j < end; ++j) pr = fmaxf(pr, p[j]);
    return pr;
  };

  // ---- load: keys and protected flags of the CTA's slice (coalesced over the block)
  if (FUSED) {
    const float* u = P.scores + (int64_t)h * bt.n_tot + q.tok_off;
    float* fo = P.fused_out + (int64_t)h * bt.m_tot + q.item_off;
    const int half = (cs == 1 && P.pool_kind != CC_POOL_NONE) ? P.pool_size / 2 : 0;
    float* us = reinterpret_cast<float*>(flags + ((kThreads * per + 15) / 16) * 16);
    if (cs == 1) {
      // stage u[cta_lo - half, cta_hi + half) (zero outside the sequence) and park the priors in
      // the key slots; four loads of each are issued before the first store, so the slice
      // costs a couple of round trips to L2 instead of one per item
      const int span = cta_items + 2 * half;
#pragma unroll 1
      for (int t0 = threadIdx.x; t0 < cta_items; t0 += 4 * kThreads) {
        float b[4];
#pragma unroll
        for (int k = 0; k < 4; ++k) b[k] = t0 + k * kThreads < cta_items ? p[cta_lo + t0 + k * kThreads] : 0.0f;
#pragma unroll
        for (int k = 0; k < 4; ++k)
          if (t0 + k * kThreads < cta_items) keys[padded(t0 + k * kThreads)] = __float_as_uint(b[k]);
      }
      pdl_wait();                                   // the scores are complete from here on
      if (P.stage_u) {
#pragma unroll 1
      for (int t0 = threadIdx.x; t0 < span; t0 += 4 * kThreads) {
        float a[4];
#pragma unroll
        for (int k = 0; k < 4; ++k) {
          const int t = t0 + k * kThreads, j = cta_lo - half + t;
          a[k] = (t < span && j >= 0 && j < q.n) ? u[j] : 0.0f;
        }
#pragma unroll
        for (int k = 0; k < 4; ++k)
          if (t0 + k * kThreads < span) us[t0 + k * kThreads] = a[k];
      }
      }
      __syncthreads();
    }
    // raw score at position t of the staged window (token cta_lo - half + t; zero outside the
    // sequence): from the staging buffer, or straight from global memory through L1 when the
    // slice is too long to be staged as well
    const bool staged = P.stage_u != 0;
    auto uval = [&](int t) -> float {
      if (staged) return us[t];
      const int j = cta_lo - half + t;
      return (j >= 0 && j < q.n) ? u[j] : 0.0f;
    };
#pragma unroll 1
    for (int li = threadIdx.x; li < cta_items; li += kThreads) {
      const int i = cta_lo + li;
      float val, pr;
      if (cs > 1) {
        // chunk sum in token order; the loads of eight tokens are issued before they are used
        const int t0 = i * cs, t1 = min(q.n, t0 + cs);
        val = 0.0f;
        pr = -INFINITY;
        for (int j0 = t0; j0 < t1; j0 += 8) {
          float a[8], b[8];
#pragma unroll
          for (int k = 0; k < 8; ++k) {
            a[k] = j0 + k < t1 ? u[j0 + k] : 0.0f;
            b[k] = j0 + k < t1 ? p[j0 + k] : -INFINITY;
          }
#pragma unroll
          for (int k = 0; k < 8; ++k) {
            if (j0 + k < t1) {
              val = (j0 + k == t0) ? a[k] : __fadd_rn(val, a[k]);
              pr = fmaxf(pr, b[k]);
            }
          }
        }
      } else {
        pr = __uint_as_float(keys[padded(li)]);       // parked by this very thread
        if (half == 0) {
          val = uval(li);
        } else if (P.pool_kind == CC_POOL_MAX) {
          val = uval(li + half);
          const int a = max(0, i - half), b = min(q.n - 1, i + half);
          for (int j = a; j <= b; ++j) val = fmaxf(val, uval(j - cta_lo + half));
        } else {
          val = uval(li);
          for (int d = 1; d <= 2 * half; ++d) val = __fadd_rn(val, uval(li + d));
          val = __fdiv_rn(val, (float)P.pool_size);
        }
      }
      const float f = __fadd_rn(__fadd_rn(__fmul_rn(P.alpha, val), __fmul_rn(P.beta, pr)), 0.0f);
      fo[i] = f;
      keys[padded(li)] = mono_key(f);
      flags[li] = pr >= theta ? 1 : 0;
    }
  } else {
    const float* f = P.fused_in + (int64_t)h * bt.m_tot + q.item_off;
#pragma unroll 1
    for (int li = threadIdx.x; li < cta_items; li += kThreads) {
      keys[padded(li)] = mono_key(f[cta_lo + li]);
      flags[li] = item_prior(li) >= theta ? 1 : 0;
    }
  }
  __syncthreads();

  // ---- stage 0: protected weight
  unsigned wf = 0, free_min = 0xffffffffu, free_max = 0u;   // key range of the unprotected items
#pragma unroll 1
  for (int li = lo; li < hi; ++li) {
    if (flags[li]) {
      wf += item_len(li);
    } else {
      const unsigned key = keys[padded(li)];
      free_min = min(free_min, key);
      free_max = max(free_max, key);
    }
  }
  // one exchange yields the sum, its prefix (all the emission needs when the protected items
  // alone fill the budget: the scan of stage 3 is skipped) and the key range of stage 2
  unsigned forced_before, forced_tokens;
  c.cluster_scan_total(wf, forced_before, forced_tokens, free_min, free_max);
  bool flags_as_counted = true;

  // ---- stage 1: cap on protected items (longest prefix by (prior desc, index asc) within B_span)
  if (q.span_cap >= 0 && forced_tokens > (unsigned)q.span_cap) {
    flags_as_counted = false;
    const unsigned cap = (unsigned)q.span_cap;
    unsigned t1, above1;
    bool whole;
    radix_threshold(c, lo, hi, cap + 1u, false,
                    [&](int li, unsigned& key, unsigned& len) {
                      if (!flags[li]) return false;
                      key = mono_key(item_prior(li));
                      len = item_len(li);
                      return true;
                    }, t1, above1, whole);
    unsigned tie_w = 0;
#pragma unroll 1
    for (int li = lo; li < hi; ++li)
      if (flags[li] && mono_key(item_prior(li)) == t1) tie_w += item_len(li);
    unsigned tie_before, dummy;
    c.cluster_scan2(tie_w, 0u, tie_before, dummy);
    unsigned kept = 0;
#pragma unroll 1
    for (int li = lo; li < hi; ++li) {
      if (!flags[li]) continue;
      const unsigned key = mono_key(item_prior(li));
      const unsigned len = item_len(li);
      if (key > t1) { kept += len; continue; }
      if (key == t1) {
        const bool fits = above1 + tie_before + len <= cap;
        tie_before += len;
        if (fits) { kept += len; continue; }
      }
      flags[li] = 0;
    }
    forced_tokens = c.cluster_sum(kept);
  }

  // ---- stage 2: cut-off among the unprotected items
  bool ties_are_forced, whole_bin = false;
  unsigned t = 0, tie_budget;
  if (forced_tokens >= keep) {
    ties_are_forced = true;          // protected items alone fill the budget: first B in order
    tie_budget = keep;
  } else {
    ties_are_forced = false;
    unsigned above;
    radix_threshold(c, lo, hi, keep - forced_tokens, true,
                    [&](int li, unsigned& key, unsigned& len) {
                      if (flags[li]) return false;
                      key = keys[padded(li)];
                      len = item_len(li);
                      return true;
                    }, t, above, whole_bin, flags_as_counted, free_min, free_max);
    tie_budget = keep - forced_tokens - above;
  }

  // ---- stage 3: ordered emission
  const bool reuse_prefix = ties_are_forced && flags_as_counted;
  unsigned def_w = 0, tie_w = 0;
  if (!reuse_prefix) {
#pragma unroll 1
  for (int li = lo; li < hi; ++li) {
    const unsigned len = item_len(li);
    if (flags[li]) {
      if (ties_are_forced) tie_w += len; else def_w += len;
    } else if (!ties_are_forced) {
      const unsigned key = keys[padded(li)];
      if (key > t || (whole_bin && key == t)) def_w += len; else if (key == t) tie_w += len;
    }
  }
  }
  unsigned def_before, tie_before;
  if (reuse_prefix) {
    def_before = 0;
    tie_before = forced_before;
  } else {
    c.cluster_scan2(def_w, tie_w, def_before, tie_before);
  }
  // last read of a peer's shared memory is done: announce it now, wait for the peers at the
  // very end, and write the indices in between
  if (c.C > 1) asm volatile("barrier.cluster.arrive.release.aligned;" ::: "memory");
#pragma unroll 1
  for (int li = lo; li < hi; ++li) {
    const unsigned len = item_len(li);
    unsigned take = 0;
    bool tie = false;
    if (flags[li]) {
      if (ties_are_forced) tie = true; else take = len;
    } else if (!ties_are_forced) {
      const unsigned key = keys[padded(li)];
      if (key > t || (whole_bin && key == t)) take = len; else if (key == t) tie = true;
    }
    const unsigned pos = def_before + min(tie_before, tie_budget);
    if (tie) {
      take = tie_before < tie_budget ? min(len, tie_budget - tie_before) : 0u;
      tie_before += len;
    } else {
      def_before += take;
    }
    const int tok0 = (cta_lo + li) * cs;
    for (unsigned k = 0; k < take; ++k)
      if (pos + k < keep) out[pos + k] = tok0 + (int)k;
  }
  for (int i = (int)keep + c.rank * kThreads + threadIdx.x; i < q.budget; i += c.C * kThreads)
    out[i] = -1;
  if (c.rank == 0 && threadIdx.x == 0) P.count[s * P.hkv + h] = (int)keep;
  // no CTA may leave while a peer can still read its shared memory
  if (c.C > 1) asm volatile("barrier.cluster.wait.acquire.aligned;" ::: "memory");
}

size_t cluster_smem_bytes(int per, bool staged, int pool_size) {
  size_t b = sizeof(Shared);
  b += ((size_t)padded(kThreads * per) + 1) * 4;          // keys
  b += ((size_t)kThreads * per + 15) / 16 * 16;           // flags
  if (staged) b += ((size_t)kThreads * per + 2 * (pool_size / 2) + 4) * 4;
  return (b + 15) / 16 * 16;
}

}  // namespace

// CTAs per (sequence, head) for the cluster kernel, or 0 when the batch does not fit.
// A CTA holds up to kCtaItems items (32 per thread; the fused form also stages the raw scores of
// slices of up to 16 per thread and reads them through L1 beyond that); one CTA of 1024 threads fits per SM, and a
// cluster is placed inside one GPC, so about 96 CTAs run at a time in clusters of eight, 128 in
// clusters of four, all 148 otherwise.  Wide clusters finish one (sequence, head) sooner, narrow
// ones let more of them run at once and pay less per exchange (measured: about 6 + 0.6 x width +
// items per thread microseconds): the width with the smallest waves x time per wave is taken.
int select_cluster_size(const BatchTable& bt, int hkv) {
  if (bt.max_items <= 0) return 1;
  // in chunk mode a thread reads all tokens of its items, so the width is chosen by tokens
  const long long work = (long long)bt.max_items * bt.chunk;
  const long long problems = (long long)bt.num_seqs * hkv;
  auto per_of = [&](int c) { return (bt.max_items + c * kThreads - 1) / (c * kThreads); };
  auto cost_of = [&](int c) {
    const long long room = c == 8 ? 96 : (c == 4 ? 128 : 148);
    const double waves = (double)((problems * c + room - 1) / room);
    return waves * (6.0 + 0.6 * c + 1.05 * (double)((work + c * kThreads - 1) / (c * kThreads)));
  };
  // widest useful cluster: four items per thread ...
  int c = 1;
  while (c < kMaxCluster && (work + c * kThreads - 1) / (c * kThreads) > 4) c *= 2;
  if (kThreads * per_of(c) > kCtaItems) return 0;
  // ... narrowed while the batch needs several waves and fewer, longer waves are cheaper
  while (c > 1 && kThreads * per_of(c / 2) <= kCtaItems && cost_of(c / 2) < cost_of(c)) c /= 2;
  return c;
}

cudaError_t launch_select_cluster(const Launch& L, const BatchTable& bt, const Geometry& g,
                                  float force_threshold, bool fused_input, int pool_kind,
                                  int pool_size, float alpha, float beta, const float* scores,
                                  float* fused, const float* prior, int32_t* idx, int32_t* count,
                                  int cluster) {
  ClusterParams P;
  P.cluster = cluster;
  P.hkv = g.hkv;
  P.theta = force_threshold;
  P.pool_kind = pool_kind;
  P.pool_size = pool_kind == CC_POOL_NONE ? 1 : pool_size;
  P.alpha = alpha;
  P.beta = beta;
  P.scores = scores;
  P.fused_out = fused;
  P.fused_in = fused;
  P.prior = prior;
  P.idx = idx;
  P.count = count;
  const int per = bt.max_items > 0 ? (bt.max_items + cluster * kThreads - 1) / (cluster * kThreads) : 1;
  // token-level fused form: stage the slice's raw scores while they fit beside keys and flags
  P.stage_u = fused_input && bt.chunk == 1 && kThreads * per <= kStagedItems ? 1 : 0;
  const size_t smem = cluster_smem_bytes(per, P.stage_u != 0, P.pool_size);
  const bool chunked = bt.chunk > 1;
  auto kern = fused_input ? (chunked ? select_cluster_kernel<true, true> : select_cluster_kernel<true, false>)
                          : (chunked ? select_cluster_kernel<false, true> : select_cluster_kernel<false, false>);
  cudaError_t e = cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
  if (e != cudaSuccess) return e;
  return launch_pdl(kern, dim3(cluster, g.hkv, bt.num_seqs), dim3(kThreads), smem, L.stream, cluster, bt, P);
}

}  // namespace cc
