// A1, tensor-core mode (CC_MODE_BF16): window attention scores on sm_100a.
//
// u_h(j) = sum_r exp(s_rj - L_r) with s = q_r . k_j / sqrt(d) and L_r = log sum_j exp(s_rj),
// where r runs over the w * G query rows that share KV head h.  L_r needs every key before
// any column can be reduced, so the keys are streamed twice with the same persistent kernel:
//
//   pass 1  S = Q K^T with query rows on the MMA M axis: one TMEM lane, hence one thread, per
//           query row, so the running maximum and sum of exp need no cross-thread traffic.
//           Each CTA covers a contiguous span of key tiles and writes one (max, sum) pair per
//           row; the spans of a (sequence, head) are merged in pass 2.
//   pass 2  S^T = K Q^T with keys on the M axis: one thread per key, the query rows along the
//           TMEM columns, so u(j) is a plain in-thread sum and is stored coalesced.
//
// Pipeline per CTA (one CTA per SM, 608 threads): warp 0 issues TMA loads (K tiles of 128 keys
// through a ring of shared-memory stages, Q once per (sequence, head)), two warps issue
// tcgen05.mma into four TMEM accumulator buffers, sixteen warps drain the accumulators with
// tcgen05.ld and do the exp / reduction work while later tiles are being multiplied.
// All operands sit in shared memory in the 128-byte-swizzled K-major layout that both TMA
// and the MMA descriptors understand; Q and K simply swap the A / B roles between passes.
//
// TMEM holds four accumulator buffers of 128 columns; work item i (one 128 x 128 block of S or
// S^T) lands in buffer i mod 4.  The sixteen epilogue warps form four sets of four (one warp
// per TMEM lane quadrant); set k drains buffer k, so every scheduler hosts one warp of each set
// and the sets run staggered: while one set waits for its buffer to be refilled, the other
// three keep the special-function unit busy.  The exponentials are the bottleneck of both
// passes (16 per clock on the special-function unit against 8192 tensor flops per clock), and
// what counts is that the unit never idles: a warp reads 32 columns at a time, so it needs few
// registers and four warps fit per scheduler; scaling and accumulation use packed f32x2
// instructions; one pair of exponentials in kPolyEvery is evaluated on the FMA pipe instead
// (round to nearest integer, degree-3 polynomial for the fraction, exponent patched in by
// integer arithmetic; relative error 8e-5).
//
// Every wait on an mbarrier is bounded: when the bound is hit the kernel records
// CC_ERR_TIMEOUT, every role leaves its loop, TMEM is released and the kernel returns.
#include <string.h>

#include <type_traits>

#include "cc_internal.cuh"
#include "exp2_poly.cuh"

namespace cc {

namespace {

#ifndef CC_ISSUERS
#define CC_ISSUERS 2
#endif
constexpr int kIssuers = CC_ISSUERS;                      // 1 or 2
constexpr int kEpiWarps = 16;
constexpr int kThreads = (1 + kIssuers + kEpiWarps) * 32; // TMA, the MMA issuers, 16 epilogue warps
constexpr int kMmaWarpB = 2 + kEpiWarps;                  // second MMA issuer (the last warp), if any
static_assert(kIssuers == 1 || kIssuers == 2, "every warp of the CTA needs a role");
static_assert(kThreads / 32 == kMmaWarpB + kIssuers - 1, "warps 0, 1, the epilogue warps, the second issuer");
constexpr int kEpiThreads = kEpiWarps * 32;
constexpr int kMaxStages = 6;
constexpr uint32_t kPanelBytes = kTileKeys * 128;        // one 64-channel half of a K tile
constexpr uint32_t kStageBytes = 2 * kPanelBytes;        // 32 KB
constexpr uint32_t kTmemCols = 512;
constexpr uint32_t kBufCols = 128;                        // accumulator buffer stride
constexpr int kBufs = 4;                                  // accumulator buffers in TMEM
constexpr int kSets = 4;                                  // epilogue warp sets, one per buffer
constexpr uint32_t kMiscBytes = 20480;
constexpr uint32_t kSmemLimit = 232448;                   // 227 KB
constexpr float kLog2e = 1.4426950408889634f;
constexpr float kLn2 = 0.6931471805599453f;

struct TcParams {
  int grid;            // CTAs (same for both passes)
  int total_tiles;     // H_kv * sum of tiles over the sequences
  int rows;            // w * G
  int rows_pad;        // G * w_pad, a multiple of 16
  int w_pad;
  int n_stages;
  int n_sub;           // pass 1: 128-row blocks; pass 2: column chunks
  int sub_cols;        // pass 2: rows per column chunk (multiple of 16, <= 128)
  float2* part;        // [(grid + problems)][rows_pad] (max, sum) in the log2 domain
  float* scores;
  float* lse;
  int64_t pool_rows;
  // K tile in shared memory.  Contiguous cache: two panels of 64 channels, each 128 rows of 128
  // bytes (8-row groups 1024 bytes apart, second panel 16 KB on).  Paged cache: one copy per page
  // lays the rows out in 8-token groups of 2 KB, first panel then second (8-row groups of a panel
  // 2048 bytes apart, second panel 1 KB on), whatever the page size.
  uint32_t k_sbo16;      // stride between 8-row groups of a panel, in 16-byte units
  uint32_t k_panel16;    // offset of the second panel, in 16-byte units
};

// ------------------------------------------------------------------ PTX wrappers
__device__ __forceinline__ uint32_t smem_u32(const void* p) {
  return (uint32_t)__cvta_generic_to_shared(p);
}
__device__ __forceinline__ void mbar_init(uint32_t bar, uint32_t count) {
  asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(bar), "r"(count) : "memory");
}
__device__ __forceinline__ void mbar_expect_tx(uint32_t bar, uint32_t bytes) {
  asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(bar), "r"(bytes)
               : "memory");
}
__device__ __forceinline__ void mbar_arrive(uint32_t bar) {
  asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(bar) : "memory");
}
// One probe of the barrier phase; the hardware may park the thread for up to the given number
// of nanoseconds while the phase is incomplete, so a waiting warp does not take issue slots
// from the warps that have work.
__device__ __forceinline__ uint32_t mbar_try_wait(uint32_t bar, uint32_t parity) {
  uint32_t ok;
  asm volatile(
      "{\n\t.reg .pred p;\n\t"
      "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2, %3;\n\t"
      "selp.u32 %0, 1, 0, p;\n\t}"
      : "=r"(ok) : "r"(bar), "r"(parity), "r"(2000u) : "memory");
  return ok;
}
__device__ __forceinline__ void fence_barrier_init() {
  asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
}
// K tile copy with an L2 eviction-priority hint: pass 1 asks L2 to keep the tile (pass 2 reads
// it again), pass 2 marks it as the first to go.
__device__ __forceinline__ void tma_load_3d_hint(uint32_t dst, const CUtensorMap* map, uint32_t bar,
                                                 int c0, int c1, int c2, uint64_t policy) {
  asm volatile(
      "cp.async.bulk.tensor.3d.shared::cluster.global.tile.mbarrier::complete_tx::bytes.L2::cache_hint "
      "[%0], [%1, {%3, %4, %5}], [%2], %6;"
      ::"r"(dst), "l"(map), "r"(bar), "r"(c0), "r"(c1), "r"(c2), "l"(policy) : "memory");
}
// One page of a paged cache: box (64 channels, 8 tokens, 2 panels, page_size / 8 groups, 1 head).
__device__ __forceinline__ void tma_load_5d_hint(uint32_t dst, const CUtensorMap* map, uint32_t bar,
                                                 int c3, int c4, uint64_t policy) {
  asm volatile(
      "cp.async.bulk.tensor.5d.shared::cluster.global.tile.mbarrier::complete_tx::bytes.L2::cache_hint "
      "[%0], [%1, {%3, %3, %3, %4, %5}], [%2], %6;"
      ::"r"(dst), "l"(map), "r"(bar), "r"(0), "r"(c3), "r"(c4), "l"(policy) : "memory");
}
__device__ __forceinline__ void tma_load_4d(uint32_t dst, const CUtensorMap* map, uint32_t bar,
                                            int c0, int c1, int c2, int c3) {
  asm volatile(
      "cp.async.bulk.tensor.4d.shared::cluster.global.tile.mbarrier::complete_tx::bytes "
      "[%0], [%1, {%3, %4, %5, %6}], [%2];"
      ::"r"(dst), "l"(map), "r"(bar), "r"(c0), "r"(c1), "r"(c2), "r"(c3) : "memory");
}
__device__ __forceinline__ void tmem_alloc(uint32_t smem_dst, uint32_t cols) {
  asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;"
               ::"r"(smem_dst), "r"(cols) : "memory");
}
__device__ __forceinline__ void tmem_relinquish() {
  asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
}
__device__ __forceinline__ void tmem_dealloc(uint32_t taddr, uint32_t cols) {
  asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(taddr), "r"(cols)
               : "memory");
}
__device__ __forceinline__ void tc_fence_before() {
  asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
}
__device__ __forceinline__ void tc_fence_after() {
  asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
}
__device__ __forceinline__ void umma_commit(uint32_t bar) {
  asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];"
               ::"r"(bar) : "memory");
}
__device__ __forceinline__ void tmem_ld32(uint32_t taddr, uint32_t (&v)[32]) {
  asm volatile(
      "tcgen05.ld.sync.aligned.32x32b.x32.b32 "
      "{%0,%1,%2,%3,%4,%5,%6,%7,%8,%9,%10,%11,%12,%13,%14,%15,"
      "%16,%17,%18,%19,%20,%21,%22,%23,%24,%25,%26,%27,%28,%29,%30,%31}, [%32];"
      : "=r"(v[0]), "=r"(v[1]), "=r"(v[2]), "=r"(v[3]), "=r"(v[4]), "=r"(v[5]), "=r"(v[6]),
        "=r"(v[7]), "=r"(v[8]), "=r"(v[9]), "=r"(v[10]), "=r"(v[11]), "=r"(v[12]), "=r"(v[13]),
        "=r"(v[14]), "=r"(v[15]), "=r"(v[16]), "=r"(v[17]), "=r"(v[18]), "=r"(v[19]), "=r"(v[20]),
        "=r"(v[21]), "=r"(v[22]), "=r"(v[23]), "=r"(v[24]), "=r"(v[25]), "=r"(v[26]), "=r"(v[27]),
        "=r"(v[28]), "=r"(v[29]), "=r"(v[30]), "=r"(v[31])
      : "r"(taddr) : "memory");
}
__device__ __forceinline__ void tmem_wait_ld() {
  asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory");
}
__device__ __forceinline__ void epi_barrier() {      // the sixteen epilogue warps only
  asm volatile("bar.sync 1, %0;" ::"n"(kEpiThreads) : "memory");
}
__device__ __forceinline__ float max3(float a, float b, float c) {
  float d;
  asm("max.f32 %0, %1, %2, %3;" : "=f"(d) : "f"(a), "f"(b), "f"(c));
  return d;
}
__device__ __forceinline__ float max32(const uint32_t (&v)[32]) {
  float m0 = max3(__uint_as_float(v[0]), __uint_as_float(v[1]), __uint_as_float(v[2]));
  float m1 = max3(__uint_as_float(v[3]), __uint_as_float(v[4]), __uint_as_float(v[5]));
#pragma unroll
  for (int i = 6; i < 30; i += 4) {
    m0 = max3(m0, __uint_as_float(v[i]), __uint_as_float(v[i + 1]));
    m1 = max3(m1, __uint_as_float(v[i + 2]), __uint_as_float(v[i + 3]));
  }
  return max3(max3(m0, m1, __uint_as_float(v[30])), __uint_as_float(v[31]), __uint_as_float(v[31]));
}

// Instruction descriptor: bf16 x bf16 -> f32, both operands K-major.
__host__ __device__ constexpr uint32_t instr_desc(uint32_t m, uint32_t n) {
  return (1u << 4) | (1u << 7) | (1u << 10) | ((n >> 3) << 17) | ((m >> 4) << 24);
}

// ------------------------------------------------------------------ shared state
struct Barriers {
  uint64_t full[kMaxStages];
  uint64_t empty[kMaxStages];
  uint64_t q_full, q_empty;
  uint64_t acc_full[kBufs], acc_empty[kBufs];
  uint64_t u_full[8][4];             // pass 2: the other sets' partial sums of (slot, quadrant)
};

struct Misc {                        // lives in the last kMiscBytes of dynamic shared memory
  float neg_lc[kMaxRows];            // pass 2: -L_r in the log2 domain (-1e4 for padded rows)
  union {
    float2 xchg[kSets][kMaxRows];    // (max, sum) hand-over: pass 1 per set, pass 2 while merging
    float u_part[8][kSets][kTileKeys];   // pass 2: partial column sums, slot = tile & 7
  };
  Barriers bar;
  uint32_t tmem_base;
  volatile int abort_flag;
};
static_assert(sizeof(Misc) <= kMiscBytes, "Misc does not fit");

struct Pipe {
  Misc* misc;
  DeviceStatus* status;
};

// Bounded wait; false (and the abort flag set) when the bound is hit or another role gave up.
// A healthy wait lasts microseconds; the bound is 50 ms of wall-clock time (the global timer is
// read only after the first probes have failed, and then once every eight probes).
__device__ __forceinline__ unsigned long long global_ns() {
  unsigned long long t;
  asm volatile("mov.u64 %0, %%globaltimer;" : "=l"(t));
  return t;
}
__device__ __noinline__ bool wait_bar(const Pipe& p, uint64_t* bar, uint32_t parity, int where) {
  const uint32_t b = smem_u32(bar);
  for (int i = 0; i < 64; ++i)
    if (mbar_try_wait(b, parity)) return true;
  const unsigned long long t0 = global_ns();
  for (;;) {
#pragma unroll 1
    for (int i = 0; i < 8; ++i) {
      if (mbar_try_wait(b, parity)) return true;
      __nanosleep(200);
    }
    if (p.misc->abort_flag) return false;
    if (global_ns() - t0 > 50ull * 1000 * 1000) break;
  }
  p.misc->abort_flag = 1;
  report_error(p.status, CC_ERR_TIMEOUT, where);
  return false;
}

// Walks the tiles of a CTA's span in (sequence, head, tile) order.
struct TileCursor {
  int s, h, local, n_tiles;
  __device__ void locate(const BatchTable& bt, int hkv, int t) {
    for (s = 0; s < bt.num_seqs; ++s) {
      const int lo = hkv * bt.seq[s].tile_off, cnt = hkv * bt.seq[s].n_tiles;
      if (t < lo + cnt) {
        n_tiles = bt.seq[s].n_tiles;
        h = (t - lo) / n_tiles;
        local = (t - lo) % n_tiles;
        return;
      }
    }
    s = bt.num_seqs - 1; h = 0; local = 0; n_tiles = 1;   // not reached for t < total_tiles
  }
  __device__ void advance(const BatchTable& bt, int hkv) {
    if (++local < n_tiles) return;
    local = 0;
    if (++h < hkv) return;
    h = 0;
    do { ++s; } while (s < bt.num_seqs && bt.seq[s].n_tiles == 0);
    n_tiles = s < bt.num_seqs ? bt.seq[s].n_tiles : 1;
  }
  __device__ int problem(int hkv) const { return s * hkv + h; }
};

__device__ __forceinline__ int span_begin(int b, const TcParams& P) {
  return (int)(((long long)b * P.total_tiles) / P.grid);
}
__device__ __forceinline__ int cta_of_tile(int t, const TcParams& P) {
  return (int)((((long long)t + 1) * P.grid - 1) / P.total_tiles);
}

// ------------------------------------------------------------------ the kernel
// CAUSAL instantiations carry the masked copies of the epilogue loops; the others have none of
// that code.
template <int PASS, bool CAUSAL>
__global__ void __launch_bounds__(kThreads, 1)
score_tc_kernel(const __grid_constant__ BatchTable bt, const __grid_constant__ Geometry g,
                const __grid_constant__ TcParams P, const __grid_constant__ CUtensorMap q_map,
                const __grid_constant__ CUtensorMap k_map, DeviceStatus* status) {
  extern __shared__ uint8_t smem_raw[];
  uint8_t* smem = reinterpret_cast<uint8_t*>(((uintptr_t)smem_raw + 1023) & ~(uintptr_t)1023);
  const uint32_t q_bytes = (uint32_t)P.rows_pad * 256u;
  const uint32_t q_panel = (uint32_t)P.rows_pad * 128u;
  uint8_t* q_smem = smem;
  uint8_t* k_smem = smem + q_bytes;
  Misc* misc = reinterpret_cast<Misc*>(k_smem + (size_t)P.n_stages * kStageBytes);
  Pipe pipe{misc, status};

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int t_begin = span_begin(blockIdx.x, P), t_end = span_begin(blockIdx.x + 1, P);

  if (threadIdx.x == 32) {
    // fetch the two TMA descriptors (kernel parameters) while the barriers are being set up
    asm volatile("prefetch.tensormap [%0];" ::"l"(reinterpret_cast<uint64_t>(&q_map)) : "memory");
    asm volatile("prefetch.tensormap [%0];" ::"l"(reinterpret_cast<uint64_t>(&k_map)) : "memory");
  }
  if (threadIdx.x == 0) {
    for (int i = 0; i < kMaxStages; ++i) {
      mbar_init(smem_u32(&misc->bar.full[i]), 1);
      mbar_init(smem_u32(&misc->bar.empty[i]), kIssuers);   // one arrival per MMA issuer
    }
    mbar_init(smem_u32(&misc->bar.q_full), 1);
    mbar_init(smem_u32(&misc->bar.q_empty), kIssuers);
    for (int i = 0; i < kBufs; ++i) {
      mbar_init(smem_u32(&misc->bar.acc_full[i]), 1);
      mbar_init(smem_u32(&misc->bar.acc_empty[i]), 4);       // the four warps of a set
    }
    for (int i = 0; i < 8; ++i)
      for (int j = 0; j < 4; ++j)        // one arrival per set that hands its partial sums over
        mbar_init(smem_u32(&misc->bar.u_full[i][j]), P.n_sub > 1 ? P.n_sub - 1 : 1);
    misc->abort_flag = 0;
    fence_barrier_init();
  }
  if (warp == 1) {
    tmem_alloc(smem_u32(&misc->tmem_base), kTmemCols);
    tmem_relinquish();
  }
  if (PASS == 2) pdl_launch_dependents();
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem_base = misc->tmem_base;
  // Pass 1 reads Q and K, which the launch before it in the stream may have produced: every
  // thread waits for that launch, and only then lets pass 2 be scheduled, so that whatever runs
  // after pass 1 has begun finds the caller's inputs complete.  The launch before pass 2 is
  // pass 1, which only produces the row statistics: the TMA and MMA roles of pass 2 start at
  // once (their first K tiles and products overlap the tail of pass 1) and only the epilogue
  // warps, which read the statistics and write the scores, wait.
  if (PASS == 1) {
    pdl_wait();
    pdl_launch_dependents();
  }

  if (warp == 0) {
    // ================================================================ TMA producer
    // The whole warp walks the tile list; lane 0 waits and issues the copies of contiguous K.
    // With a paged cache every lane owns one page of the tile: it reads the page id (before the
    // wait for the stage, so the load is covered), checks it and issues the two copies of its
    // page, so the page-table look-ups of a tile are one parallel load instead of a chain.
    {
      TileCursor cur;
      cur.locate(bt, g.hkv, t_begin);
      int stage = 0, cur_problem = -1;
      uint32_t phase = 0, qe_phase = 0;
      const int ps = bt.page_size;
      uint64_t k_policy;
      if (PASS == 1) asm volatile("createpolicy.fractional.L2::evict_last.b64 %0, 1.0;" : "=l"(k_policy));
      else           asm volatile("createpolicy.fractional.L2::evict_first.b64 %0, 1.0;" : "=l"(k_policy));
      for (int t = t_begin; t < t_end; ++t, cur.advance(bt, g.hkv)) {
        const SeqInfo& sq = bt.seq[cur.s];
        if (cur.problem(g.hkv) != cur_problem) {
          if (cur_problem >= 0) {
            const bool got = lane != 0 || wait_bar(pipe, &misc->bar.q_empty, qe_phase, 10);
            if (!__all_sync(0xffffffffu, got)) break;
            qe_phase ^= 1;
          }
          cur_problem = cur.problem(g.hkv);
          if (lane == 0) {
            const uint32_t qb = smem_u32(&misc->bar.q_full);
            mbar_expect_tx(qb, q_bytes);
            tma_load_4d(smem_u32(q_smem), &q_map, qb, 0, cur.h * g.group, 0, cur.s);
            tma_load_4d(smem_u32(q_smem) + q_panel, &q_map, qb, 64, cur.h * g.group, 0, cur.s);
          }
        }
        const int key0 = cur.local * kTileKeys;
        int page_id = -1;
        bool mine = false;               // this lane owns a page of the tile
        if (ps > 0) {
          const int valid = min(kTileKeys, sq.n - key0);
          mine = lane < (valid + ps - 1) / ps;
          if (mine) page_id = g.page_table[(int64_t)cur.s * g.page_table_stride + key0 / ps + lane];
        }
        {
          const bool got = lane != 0 || wait_bar(pipe, &misc->bar.empty[stage], phase ^ 1, 11);
          if (!__all_sync(0xffffffffu, got)) break;
        }
        const uint32_t fb = smem_u32(&misc->bar.full[stage]);
        const uint32_t dst = smem_u32(k_smem) + (uint32_t)stage * kStageBytes;
        if (ps == 0) {
          if (lane == 0) {
            mbar_expect_tx(fb, kStageBytes);
            tma_load_3d_hint(dst, &k_map, fb, 0, cur.h, sq.tok_off + key0, k_policy);
            tma_load_3d_hint(dst + kPanelBytes, &k_map, fb, 64, cur.h, sq.tok_off + key0, k_policy);
          }
        } else {
          const bool good = mine && page_id >= 0 && ((int64_t)page_id + 1) * ps <= P.pool_rows;
          if (mine && !good) report_error(status, CC_ERR_DEVICE_FLAG, 12);
          const unsigned good_mask = __ballot_sync(0xffffffffu, good);
          // the stage completes when the bytes of the good pages have landed; the expectation is
          // registered before any lane issues a copy
          if (lane == 0) mbar_expect_tx(fb, (uint32_t)__popc(good_mask) * (uint32_t)ps * 256u);
          __syncwarp();
          if (good)      // the page's rows, both panels, in one copy
            tma_load_5d_hint(dst + (uint32_t)lane * (uint32_t)ps * 256u, &k_map, fb,
                             page_id * (ps >> 3), cur.h, k_policy);
        }
        if (++stage == P.n_stages) { stage = 0; phase ^= 1; }
      }
    }
  } else if (warp == 1 || (kIssuers == 2 && warp == kMmaWarpB)) {
    // ================================================================ MMA issuers
    // The serial instruction stream of a thread that issues tcgen05.mma (waits, descriptor
    // words, eight multiplications and a commit per item) is long, so there are two issuers;
    // items go to them in pairs (0, 1 -> first; 2, 3 -> second; ...); both wait for every K
    // tile and both hand it back.  Descriptors are formed by adding small constants
    // to a base word, the accumulate flag is a compile-time predicate, and the tile bookkeeping
    // is a countdown instead of a cursor walk.
    const int my_half = warp == 1 ? 0 : 1;
    if (lane == 0) {
      TileCursor cur;
      cur.locate(bt, g.hkv, t_begin);
      int left = cur.n_tiles - cur.local;          // tiles of the current (sequence, head) still to do
      int stage = 0;
      uint32_t phase = 0, qf_phase = 0, item = 0;
      bool need_q = true;
      // descriptor words: low = start address >> 4 | LBO field, high = SBO 1024 B, version 1,
      // 128-byte swizzle
      const uint32_t q_hi = (1024u >> 4) | (1u << 14) | (2u << 29);
      const uint32_t k_hi = P.k_sbo16 | (1u << 14) | (2u << 29);
      const uint32_t a_hi = PASS == 1 ? q_hi : k_hi, b_hi = PASS == 1 ? k_hi : q_hi;
      const uint32_t q_lo0 = ((smem_u32(q_smem) & 0x3FFFFu) >> 4) | (1u << 16);
      const uint32_t k_lo0 = ((smem_u32(k_smem) & 0x3FFFFu) >> 4) | (1u << 16);
      const uint32_t q_panel16 = q_panel >> 4;
      const uint32_t q_step16 = PASS == 1 ? (128u * 128u) >> 4 : ((uint32_t)P.sub_cols * 128u) >> 4;
      const uint32_t idesc_full =
          PASS == 1 ? instr_desc(128, kTileKeys) : instr_desc(128, (uint32_t)P.sub_cols);
      const uint32_t idesc_last =
          PASS == 1 ? idesc_full
                    : instr_desc(128, (uint32_t)(P.rows_pad - (P.n_sub - 1) * P.sub_cols));
      const uint32_t full0 = smem_u32(&misc->bar.full[0]), empty0 = smem_u32(&misc->bar.empty[0]);
      const uint32_t accf0 = smem_u32(&misc->bar.acc_full[0]);
      const uint32_t acce0 = smem_u32(&misc->bar.acc_empty[0]);
      bool ok = true;
      for (int t = t_begin; t < t_end && ok; ++t) {
        if (need_q) {
          if (!wait_bar(pipe, &misc->bar.q_full, qf_phase, 20)) break;
          qf_phase ^= 1;
          need_q = false;
        }
        if (!mbar_try_wait(full0 + 8u * (uint32_t)stage, phase) &&
            !wait_bar(pipe, &misc->bar.full[stage], phase, 21))
          break;
        tc_fence_after();
        const uint32_t k_lo = k_lo0 + (uint32_t)stage * (kStageBytes >> 4);
#pragma unroll 1
        for (int sub = 0; sub < P.n_sub; ++sub, ++item) {
          if (kIssuers == 2 && (int)((item >> 1) & 1u) != my_half) continue;
          const uint32_t buf = item & (kBufs - 1);
          const uint32_t par = ((item >> 2) & 1u) ^ 1u;
          if (!mbar_try_wait(acce0 + 8u * buf, par) &&
              !wait_bar(pipe, &misc->bar.acc_empty[buf], par, 22)) {
            ok = false;
            break;
          }
          tc_fence_after();
          const uint32_t d_tmem = tmem_base + buf * kBufCols;
          const uint32_t idesc = sub == P.n_sub - 1 ? idesc_last : idesc_full;
          const uint32_t q_lo = q_lo0 + (uint32_t)sub * q_step16;
#pragma unroll
          for (int ks = 0; ks < kHeadDim / 16; ++ks) {
            const uint32_t ql = q_lo + (ks >= 4 ? q_panel16 : 0u) + (uint32_t)(ks & 3) * 2u;
            const uint32_t kl = k_lo + (ks >= 4 ? P.k_panel16 : 0u) + (uint32_t)(ks & 3) * 2u;
            const uint32_t al = PASS == 1 ? ql : kl, bl = PASS == 1 ? kl : ql;
            if (ks == 0) {
              asm volatile(
                  "{\n\t.reg .pred p;\n\t.reg .b64 a, b;\n\tsetp.ne.b32 p, 0, 0;\n\t"
                  "mov.b64 a, {%1, %3};\n\tmov.b64 b, {%2, %5};\n\t"
                  "tcgen05.mma.cta_group::1.kind::f16 [%0], a, b, %4, p;\n\t}"
                  ::"r"(d_tmem), "r"(al), "r"(bl), "r"(a_hi), "r"(idesc), "r"(b_hi) : "memory");
            } else {
              asm volatile(
                  "{\n\t.reg .pred p;\n\t.reg .b64 a, b;\n\tsetp.eq.b32 p, 0, 0;\n\t"
                  "mov.b64 a, {%1, %3};\n\tmov.b64 b, {%2, %5};\n\t"
                  "tcgen05.mma.cta_group::1.kind::f16 [%0], a, b, %4, p;\n\t}"
                  ::"r"(d_tmem), "r"(al), "r"(bl), "r"(a_hi), "r"(idesc), "r"(b_hi) : "memory");
            }
          }
          umma_commit(accf0 + 8u * buf);
        }
        if (!ok) break;
        umma_commit(empty0 + 8u * (uint32_t)stage);
        if (++stage == P.n_stages) { stage = 0; phase ^= 1; }
        if (--left == 0 && t + 1 < t_end) {
          // the next tile belongs to another (sequence, head): Q may be replaced once the
          // multiplications issued so far have read it
          umma_commit(smem_u32(&misc->bar.q_empty));
          cur.local = cur.n_tiles - 1;
          cur.advance(bt, g.hkv);
          left = cur.n_tiles;
          need_q = true;
        }
      }
    }
  } else if (warp >= 2 && warp < 2 + kEpiWarps) {
    // ================================================================ epilogue warps
    const int ew = warp - 2;                 // 0..15
    const int quad = warp & 3;               // TMEM lane quadrant this warp may read
    const int set = ew >> 2;                 // consecutive warps cover the four quadrants
    const int row_in_tile = quad * 32 + lane;
    const int etid = ew * 32 + lane;         // 0..511, unique per epilogue thread
    const uint32_t lane_addr = tmem_base + ((uint32_t)(quad * 32) << 16);
    const float c = kLog2e / sqrtf((float)kHeadDim);
    const uint64_t c2 = pack2(c, c);
    TileCursor cur;
    cur.locate(bt, g.hkv, t_begin);
    int cur_problem = -1;
    bool dead = false;      // after a failed wait: keep the loop structure (and its barriers), skip the work
    float run_m[4] = {-INFINITY, -INFINITY, -INFINITY, -INFINITY};
    float run_l[4] = {0.f, 0.f, 0.f, 0.f};

    // pass 1: merge the four sets' (max, sum) of every row and write the span's partial
    auto flush_partial = [&](int problem) {
#pragma unroll
      for (int rb = 0; rb < 4; ++rb) {
        if (rb >= P.n_sub) break;
        // a set whose row block never changes keeps its state in slot 0
        const int own = P.n_sub == 3 ? rb : (rb == set % P.n_sub ? 0 : -1);
        float2 st = make_float2(-INFINITY, 0.f);
#pragma unroll
        for (int k = 0; k < 4; ++k) if (k == own) st = make_float2(run_m[k], run_l[k]);
        misc->xchg[set][rb * 128 + row_in_tile] = st;
      }
#pragma unroll
      for (int k = 0; k < 4; ++k) { run_m[k] = -INFINITY; run_l[k] = 0.f; }
      epi_barrier();
      for (int row = etid; row < P.rows_pad; row += kEpiThreads) {
        float m = -INFINITY;
#pragma unroll
        for (int k = 0; k < kSets; ++k) m = fmaxf(m, misc->xchg[k][row].x);
        float l = 0.f;
#pragma unroll
        for (int k = 0; k < kSets; ++k) {
          const float2 o = misc->xchg[k][row];
          if (o.y > 0.f) l += o.y * ex2(o.x - m);
        }
        P.part[(int64_t)(blockIdx.x + problem) * P.rows_pad + row] = make_float2(m, l);
      }
      epi_barrier();
    };

    // pass 2 (first_tile = the (sequence, head)'s first tile, tb = its first tile in this span):
    auto merge_lse = [&](const SeqInfo& sq, int first_tile, int tb) {
      // merge the spans' (max, sum) of the new (sequence, head) into -L_r: the spans are
      // dealt round-robin to the threads that share a row, all loads of a thread are issued
      // before the first use, and the threads of a row meet through shared memory
      epi_barrier();
      const int b0 = cta_of_tile(first_tile, P), b1 = cta_of_tile(first_tile + sq.n_tiles - 1, P);
      const int problem = cur.problem(g.hkv);
      const int ways = max(1, min(4, kEpiThreads / P.rows_pad));    // threads per row
      const int per_sweep = kEpiThreads / ways;                     // rows per sweep
      float2* fold = &misc->xchg[0][0];          // no tile is in flight here, the union is free
      for (int base = 0; base < P.rows_pad; base += per_sweep) {
        const int row = base + etid % per_sweep, way = etid / per_sweep;
        float m = -INFINITY, l = 0.f;
        if (row < P.rows_pad) {
          for (int b = b0 + way; b <= b1; b += 8 * ways) {
            float2 pr[8];
#pragma unroll
            for (int k = 0; k < 8; ++k) {
              const int bb = b + k * ways;
              pr[k] = bb <= b1 ? P.part[(int64_t)(bb + problem) * P.rows_pad + row]
                               : make_float2(-INFINITY, 0.f);
            }
#pragma unroll
            for (int k = 0; k < 8; ++k) {
              if (pr[k].y > 0.f) {
                const float mn = fmaxf(m, pr[k].x);
                l = l * ex2(m - mn) + pr[k].y * ex2(pr[k].x - mn);
                m = mn;
              }
            }
          }
          if (ways > 1) fold[etid] = make_float2(m, l);
        }
        if (ways > 1) epi_barrier();
        if (row < P.rows_pad && way == 0) {
          for (int k = 1; k < ways; ++k) {
            const float2 o = fold[k * per_sweep + etid];
            if (o.y > 0.f) {
              const float mn = fmaxf(m, o.x);
              l = l * ex2(m - mn) + o.y * ex2(o.x - mn);
              m = mn;
            }
          }
          const float lc = m + log2f(l);
          const int gq = row % g.group, tq = row / g.group;     // row = t * G + g
          const bool real = tq < g.window;
          misc->neg_lc[row] = real ? -lc : -1.0e4f;
          if (real && P.lse != nullptr && tb == first_tile)
            P.lse[((int64_t)cur.s * g.hq + cur.h * g.group + gq) * g.window + tq] = lc * kLn2;
        }
        if (ways > 1) epi_barrier();
      }
      epi_barrier();
    };

    // A set works on every fourth item of the span, item = (tile - t_begin) * n_sub + sub, and
    // steps from one of its items to the next by a precomputed (tiles, subs) stride; the
    // cursor is walked only where the (sequence, head) changes.  Buffer = set, and the phase
    // of its barrier flips with every item.
    const int n_sub = P.n_sub;
    const int dt = kSets / n_sub, ds = kSets % n_sub;
    const bool rotating = ds != 0;          // the set's row block changes from item to item
    int sub = set % n_sub, t = t_begin + set / n_sub;
    uint32_t par = 0;
    int prob_end = t_begin, first_tile = 0, n_cur = 0;
    int64_t out_base = 0;
    const uint32_t full_bar = smem_u32(&misc->bar.acc_full[set]);
    const uint32_t empty_bar = smem_u32(&misc->bar.acc_empty[set]);
    const uint32_t acc_addr = lane_addr + (uint32_t)set * kBufCols;
    if (PASS == 2) pdl_wait();
    for (;;) {
      if (t >= prob_end) {
        bool done = false;
        do {
          if (PASS == 1 && cur_problem >= 0) flush_partial(cur_problem);
          if (prob_end >= t_end) { done = true; break; }
          if (cur_problem >= 0) {
            cur.local = cur.n_tiles - 1;
            cur.advance(bt, g.hkv);
          }
          const SeqInfo& sq = bt.seq[cur.s];
          first_tile = g.hkv * sq.tile_off + cur.h * sq.n_tiles;
          if (PASS == 2) merge_lse(sq, first_tile, prob_end);
          cur_problem = cur.problem(g.hkv);
          prob_end = min(t_end, first_tile + sq.n_tiles);
          n_cur = sq.n;
          out_base = (int64_t)cur.h * bt.n_tot + sq.tok_off;
        } while (t >= prob_end);
        if (done) break;
      }
      const int key0 = (t - first_tile) * kTileKeys;
      const int valid = min(kTileKeys, n_cur - key0);
      if (!dead) {
        // every lane probes once; only when the buffer is not full yet does one lane wait
        if (!__all_sync(0xffffffffu, mbar_try_wait(full_bar, par))) {
          const bool got = lane != 0 || wait_bar(pipe, &misc->bar.acc_full[set], par, 30);
          dead = !__all_sync(0xffffffffu, got);
        }
      }
      par ^= 1u;
      float u_acc = 0.f;
      if (!dead) {
        tc_fence_after();
        uint64_t acc[4] = {0ull, 0ull, 0ull, 0ull};
        uint32_t v[32];
        if (PASS == 1) {
          // thread = query row (sub * 128 + row_in_tile); columns = the 128 keys of the tile
          float m_run = run_m[0], l_run = run_l[0];
          if (rotating) {
#pragma unroll
            for (int rb = 1; rb < 4; ++rb) if (rb == sub) { m_run = run_m[rb]; l_run = run_l[rb]; }
          }
          // keys of the tile this row attends to: all valid ones, or (causal window) those up
          // to the row's own position n - w + t
          // (the masked form is a copy of the loop of its own, so that the common one stays lean)
          const bool masked_tile = CAUSAL && key0 + kTileKeys > n_cur - g.window + 1;
          auto drain = [&](auto masked) {
          constexpr bool kMasked = decltype(masked)::value;
          // a warp whose 32 rows all lie past the padded window (last row block of a row count
          // that is not a multiple of 128) has nothing to sum: it only hands the buffer back
          int valid_r = sub * 128 + quad * 32 >= P.rows_pad ? 0 : valid;
          if (kMasked) {
            const int t_row = (sub * 128 + row_in_tile) / g.group;
            if (t_row < g.window) valid_r = min(valid, n_cur - g.window + t_row + 1 - key0);
          }
          // all 128 keys of the tile count for every row of the warp: no per-chunk range tests
          const bool full_tile = !kMasked && __shfl_sync(0xffffffffu, valid_r, 0) == kTileKeys;
#pragma unroll 1
          for (int cc0 = 0; cc0 < kTileKeys; cc0 += 32) {
            if (kMasked) __syncwarp();            // rows of a masked tile skip different chunks
            tmem_ld32(acc_addr + (uint32_t)cc0, v);
            tmem_wait_ld();
            if (cc0 + 32 == kTileKeys) {             // last read of the buffer: hand it back
              tc_fence_before();
              __syncwarp();
              if (lane == 0) mbar_arrive(empty_bar);
            }
            if (!full_tile) {
              if (cc0 >= valid_r) continue;
              if (cc0 + 32 > valid_r) {
#pragma unroll
                for (int i = 0; i < 32; ++i)
                  if (cc0 + i >= valid_r) v[i] = 0xc61c4000u;  // -1e4: its exponential underflows to 0
              }
            }
            // The reference of the exponentials only has to be near the row maximum, not equal
            // to it: it is replaced when a value lies more than 2^64 above it.  The test is a
            // warp vote where the warp is converged, so that the common case is one uniform branch.
            const float mx = max32(v) * c;
            const bool renew = m_run == -INFINITY || mx > m_run + 64.0f;
            // (the rows of a masked tile skip different chunks, so its lanes are not converged
            // here and must not vote; everywhere else the warp takes this path as one)
            if (kMasked ? renew : __any_sync(0xffffffffu, renew)) {
              if (renew) {
                if (m_run > -INFINITY) l_run = (l_run + acc_total(acc)) * ex2(m_run - mx);
                acc[0] = acc[1] = acc[2] = acc[3] = 0ull;
                m_run = mx;
              }
            }
            exp_accumulate<false, 32>(v, c2, pack2(-m_run, -m_run), 0u, acc);
          }
          };
          if (CAUSAL && masked_tile) drain(std::true_type{}); else drain(std::false_type{});
          l_run += acc_total(acc);
          if (rotating) {
#pragma unroll
            for (int rb = 0; rb < 4; ++rb) if (rb == sub) { run_m[rb] = m_run; run_l[rb] = l_run; }
          } else {
            run_m[0] = m_run;
            run_l[0] = l_run;
          }
        } else {
          // thread = key (key0 + row_in_tile); columns = the query rows of this chunk
          const int c0 = sub * P.sub_cols;
          const int nc = min(P.sub_cols, P.rows_pad - c0);        // multiple of 16
          const uint32_t nl = smem_u32(misc->neg_lc + c0);         // -L_r of the item's columns
          // causal window: key j is seen by the rows t >= j - (n - w), i.e. by the columns
          // from G * (j - n + w) on; the columns before it contribute nothing
          const bool masked_tile = CAUSAL && key0 + kTileKeys > n_cur - g.window + 1;
          auto drain = [&](auto masked) {
          constexpr bool kMasked = decltype(masked)::value;
          const int first_col = kMasked ? g.group * (key0 + row_in_tile - n_cur + g.window) : 0;
#pragma unroll 1
          for (int cc0 = 0; cc0 < nc; cc0 += 32) {
            if (kMasked) __syncwarp();
            tmem_ld32(acc_addr + (uint32_t)cc0, v);               // stays inside the 128-column buffer
            tmem_wait_ld();
            if (kMasked && first_col > c0 + cc0) {
#pragma unroll
              for (int i = 0; i < 32; ++i)
                if (c0 + cc0 + i < first_col) v[i] = 0xc61c4000u;   // -1e4: exponential ~ 0
            }
            if (cc0 + 32 >= nc) {
              tc_fence_before();
              __syncwarp();
              if (lane == 0) mbar_arrive(empty_bar);
            }
            if (cc0 + 32 <= nc) exp_accumulate<true, 32>(v, c2, 0ull, nl + 4u * (uint32_t)cc0, acc);
            else                exp_accumulate<true, 16>(v, c2, 0ull, nl + 4u * (uint32_t)cc0, acc);
          }
          };
          if (CAUSAL && masked_tile) drain(std::true_type{}); else drain(std::false_type{});
          u_acc = acc_total(acc);
        }
      }
      if (PASS == 2) {
        if (n_sub > 1) {
          // The sets that hold partial sums of the tile (one per item) meet through shared
          // memory: the set that drained the tile's last item adds the others' sums and stores;
          // n_sub - 1 arrivals complete a (slot, quadrant).  Eight slots: a slot is written
          // again only after the accumulator hand-shake has forced the reader past the tile it
          // belongs to.
          const int slot = t & 7;
          if (sub != n_sub - 1) {
            misc->u_part[slot][sub][row_in_tile] = u_acc;
            __syncwarp();
            if (lane == 0) mbar_arrive(smem_u32(&misc->bar.u_full[slot][quad]));
          } else {
            if (!dead) {
              const bool got = lane != 0 || wait_bar(pipe, &misc->bar.u_full[slot][quad],
                                                     (uint32_t)((t - t_begin) >> 3) & 1u, 31);
              dead = !__all_sync(0xffffffffu, got);
            }
            if (!dead && row_in_tile < valid) {
              float u = u_acc;
              for (int k = 0; k < n_sub - 1; ++k) u += misc->u_part[slot][k][row_in_tile];
              P.scores[out_base + key0 + row_in_tile] = u;
            }
          }
        } else if (!dead && row_in_tile < valid) {
          P.scores[out_base + key0 + row_in_tile] = u_acc;
        }
      }
      sub += ds;
      t += dt;
      if (sub >= n_sub) { sub -= n_sub; ++t; }
    }
  }

  // ---------------------------------------------------------------- teardown
  if (misc->abort_flag) {
    // give copies still in flight time to land before shared memory is released
#pragma unroll 1
    for (int i = 0; i < 2000; ++i) __nanosleep(1000);
  }
  tc_fence_before();
  __syncthreads();
  if (warp == 1) {
    tc_fence_after();
    tmem_dealloc(tmem_base, kTmemCols);
  }
}

typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*,
                                  const cuuint64_t*, const cuuint64_t*, const cuuint32_t*,
                                  const cuuint32_t*, CUtensorMapInterleave, CUtensorMapSwizzle,
                                  CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

struct TcPlan {
  TcParams P;
  size_t smem_bytes;
  bool ok;
};

TcPlan make_plan(const BatchTable& bt, const Geometry& g, int sm_count) {
  TcPlan pl;
  TcParams& P = pl.P;
  memset(&pl, 0, sizeof(pl));
  P.total_tiles = g.hkv * bt.tiles_per_head;
  P.grid = P.total_tiles < sm_count ? P.total_tiles : sm_count;
  if (P.grid < 1) P.grid = 1;
  P.rows = g.rows;
  // pad the window so that the padded row count is a multiple of 16 (UMMA N granularity)
  int w_pad = g.window;
  while ((g.group * w_pad) % 16 != 0) ++w_pad;
  P.w_pad = w_pad;
  P.rows_pad = g.group * w_pad;
  pl.ok = P.rows_pad <= kMaxRows && w_pad <= 256 && g.group <= 256;
  const uint32_t q_bytes = (uint32_t)P.rows_pad * 256u;
  int stages = ((int)kSmemLimit - 1024 - (int)kMiscBytes - (int)q_bytes) / (int)kStageBytes;
  if (stages > kMaxStages) stages = kMaxStages;
  if (stages < 2) pl.ok = false;
  P.n_stages = stages;
  pl.smem_bytes = 1024 + q_bytes + (size_t)stages * kStageBytes + kMiscBytes;
  return pl;
}

}  // namespace

size_t score_tc_ws_bytes(const BatchTable& bt, const Geometry& g, int sm_count) {
  TcPlan pl = make_plan(bt, g, sm_count);
  const size_t entries = (size_t)pl.P.grid + (size_t)bt.num_seqs * g.hkv;
  return (entries * pl.P.rows_pad * sizeof(float2) + 255) / 256 * 256;
}

cudaError_t launch_score_tc(const Launch& L, const BatchTable& bt, const Geometry& g,
                            const void* q, const void* k, float* scores, float* lse, void* ws,
                            void* encode_fn, int64_t pool_rows, int* drv_err) {
  *drv_err = 0;
  TcPlan pl = make_plan(bt, g, L.sm_count);
  if (!pl.ok) return cudaErrorInvalidConfiguration;
  TcParams& P = pl.P;
  P.part = (float2*)ws;
  P.scores = scores;
  P.lse = lse;
  P.pool_rows = bt.page_size > 0 ? pool_rows : (int64_t)bt.n_tot;

  EncodeTiledFn encode = (EncodeTiledFn)encode_fn;
  CUtensorMap q_map, k_map;
  {
    const int S = bt.num_seqs;
    cuuint64_t dims[4] = {(cuuint64_t)kHeadDim, (cuuint64_t)g.hq, (cuuint64_t)g.window, (cuuint64_t)S};
    int64_t seq_stride = g.q_stride_seq;
    if (S == 1 || seq_stride <= 0) seq_stride = g.q_stride_row * g.window;
    cuuint64_t strides[3] = {(cuuint64_t)g.q_stride_head * 2, (cuuint64_t)g.q_stride_row * 2,
                             (cuuint64_t)seq_stride * 2};
    cuuint32_t box[4] = {64, (cuuint32_t)g.group, (cuuint32_t)P.w_pad, 1};
    cuuint32_t estr[4] = {1, 1, 1, 1};
    CUresult r = encode(&q_map, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 4, const_cast<void*>(q), dims,
                        strides, box, estr, CU_TENSOR_MAP_INTERLEAVE_NONE,
                        CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                        CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
    if (r != CUDA_SUCCESS) { *drv_err = (int)r; return cudaErrorUnknown; }
  }
  if (bt.page_size > 0) {
    // A page (page_size tokens, a multiple of 8, starting at a multiple of 8 rows) as one box: 64
    // channels x 8 tokens x 2 panels x page_size / 8 groups of one head.  In shared memory that is
    // page_size / 8 blocks of 2 KB, each the eight rows of the first panel followed by the eight
    // rows of the second: two copies per page become one (a 16-token page: 4 KB per copy).
    cuuint64_t dims[5] = {64, 8, 2, (cuuint64_t)(P.pool_rows / 8), (cuuint64_t)g.hkv};
    cuuint64_t strides[4] = {(cuuint64_t)g.kv_stride_tok * 2, 128, (cuuint64_t)g.kv_stride_tok * 16,
                             (cuuint64_t)g.kv_stride_head * 2};
    cuuint32_t box[5] = {64, 8, 2, (cuuint32_t)(bt.page_size / 8), 1};
    cuuint32_t estr[5] = {1, 1, 1, 1, 1};
    CUresult r = encode(&k_map, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 5, const_cast<void*>(k), dims,
                        strides, box, estr, CU_TENSOR_MAP_INTERLEAVE_NONE,
                        CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                        CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
    if (r != CUDA_SUCCESS) { *drv_err = (int)r; return cudaErrorUnknown; }
    P.k_sbo16 = 2048u >> 4;
    P.k_panel16 = 1024u >> 4;
  } else {
    cuuint64_t dims[3] = {(cuuint64_t)kHeadDim, (cuuint64_t)g.hkv, (cuuint64_t)P.pool_rows};
    cuuint64_t strides[2] = {(cuuint64_t)g.kv_stride_head * 2, (cuuint64_t)g.kv_stride_tok * 2};
    cuuint32_t box[3] = {64, 1, (cuuint32_t)kTileKeys};
    cuuint32_t estr[3] = {1, 1, 1};
    CUresult r = encode(&k_map, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 3, const_cast<void*>(k), dims,
                        strides, box, estr, CU_TENSOR_MAP_INTERLEAVE_NONE,
                        CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                        CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
    if (r != CUDA_SUCCESS) { *drv_err = (int)r; return cudaErrorUnknown; }
    P.k_sbo16 = 1024u >> 4;
    P.k_panel16 = kPanelBytes >> 4;
  }

  auto pass1 = g.causal ? score_tc_kernel<1, true> : score_tc_kernel<1, false>;
  auto pass2 = g.causal ? score_tc_kernel<2, true> : score_tc_kernel<2, false>;
  cudaError_t e;
  e = cudaFuncSetAttribute(pass1, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)pl.smem_bytes);
  if (e != cudaSuccess) return e;
  e = cudaFuncSetAttribute(pass2, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)pl.smem_bytes);
  if (e != cudaSuccess) return e;

  P.n_sub = (P.rows_pad + 127) / 128;
  P.sub_cols = 0;
  e = launch_pdl(pass1, dim3(P.grid), dim3(kThreads), pl.smem_bytes, L.stream, 1, bt, g, P, q_map,
                 k_map, L.status);
  if (e != cudaSuccess) return e;

  P.n_sub = (P.rows_pad + 127) / 128;
  P.sub_cols = ((P.rows_pad + P.n_sub - 1) / P.n_sub + 15) / 16 * 16;
  return launch_pdl(pass2, dim3(P.grid), dim3(kThreads), pl.smem_bytes, L.stream, 1, bt, g, P, q_map,
                    k_map, L.status);
}

}  // namespace cc
