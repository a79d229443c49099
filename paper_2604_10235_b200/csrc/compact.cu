// A5: gather the retained K/V rows of every KV head into the compacted cache.
// Pure data movement: one 256-byte row of K and one of V per (slot, head), moved as
// 16-byte vectors by 16 consecutive threads, so every warp reads and writes two whole rows.
#include "cc_internal.cuh"

#include <limits.h>

namespace cc {

namespace {

constexpr int kThreads = 256;
constexpr int kLanesPerRow = kHeadDim * 2 / 16;   // 16 threads x 16 B = one bf16 row
constexpr int kRowsPerBlock = kThreads / kLanesPerRow;

__device__ __forceinline__ uint4 ld_stream(const uint4* p) {
  uint4 v;
  asm volatile("ld.global.nc.L1::no_allocate.v4.u32 {%0,%1,%2,%3}, [%4];"
               : "=r"(v.x), "=r"(v.y), "=r"(v.z), "=r"(v.w) : "l"(p));
  return v;
}
__device__ __forceinline__ void st_stream(uint4* p, uint4 v) {
  asm volatile("st.global.cs.v4.u32 [%0], {%1,%2,%3,%4};"
               :: "l"(p), "r"(v.x), "r"(v.y), "r"(v.z), "r"(v.w) : "memory");
}

// A group of 16 threads owns a unit = (slot, run of heads_per_group consecutive heads): the
// destination rows of a unit are adjacent, its page look-up on the output side is done once, and
// no division by the head count is needed (units per slot = 1 << hc_shift).  The rows of a unit
// are moved kUnroll at a time: indices first, then page entries, then the 2 * kUnroll row loads,
// then the stores.
// grid: one block per kRowsPerBlock units of a sequence, the sequences' blocks one after the
// other (a sequence without retained tokens still gets one block, which writes its page-table row)
template <int kUnroll>
__global__ void __launch_bounds__(kThreads)
compact_kernel(const __grid_constant__ BatchTable bt, const Geometry g,
               const uint16_t* __restrict__ k, const uint16_t* __restrict__ v,
               const int32_t* __restrict__ idx, uint16_t* __restrict__ k_out,
               uint16_t* __restrict__ v_out, const int32_t* __restrict__ free_pages,
               int32_t* __restrict__ out_page_table, DeviceStatus* status,
               int heads_per_group, int hc_shift) {
  pdl_launch_dependents();
  pdl_wait();
  int s = 0, local = blockIdx.x;              // sequence of this block, block index within it
  for (; s < bt.num_seqs - 1; ++s) {
    const int nb = max(1, ((bt.seq[s].keep << hc_shift) + kRowsPerBlock - 1) / kRowsPerBlock);
    if (local < nb) break;
    local -= nb;
  }
  const SeqInfo& q = bt.seq[s];
  const int lane = threadIdx.x % kLanesPerRow;
  const int grp = threadIdx.x / kLanesPerRow;
  const int ps = bt.page_size;
  // page sizes are powers of two in practice: shifts instead of divisions then
  const int ps_shift = (ps > 0 && (ps & (ps - 1)) == 0) ? __ffs(ps) - 1 : -1;

  // the block with index 0 of each sequence also publishes the sequence's new page table
  if (ps > 0 && local == 0) {
    const int used = (q.keep + ps - 1) / ps;
    for (int i = threadIdx.x; i < g.out_page_table_stride; i += kThreads) {
      int page = i < used ? free_pages[q.out_page_off + i] : -1;
      if (i < used && (page < 0 || page >= g.pool_pages)) {     // never published, never written
        report_error(status, CC_ERR_DEVICE_FLAG, 503);
        page = -1;
      }
      out_page_table[(int64_t)s * g.out_page_table_stride + i] = page;
    }
  }

  const int units = q.keep << hc_shift;          // fits: keep * heads indexes an int32 array
  const int hc_mask = (1 << hc_shift) - 1;
  const int64_t head_step = ps == 0 ? g.out_stride_head : g.kv_stride_head;
  const int32_t* pt = ps > 0 ? g.page_table + (int64_t)s * g.page_table_stride : nullptr;
  const int u = local * kRowsPerBlock + grp;
  if (u < units) {
    const int slot = u >> hc_shift;
    const int h0 = (u & hc_mask) * heads_per_group;
    int64_t dst0;                                  // destination row of (slot, head 0)
    if (ps == 0) {
      dst0 = ((int64_t)q.idx_off + slot) * g.out_stride_tok;
    } else {
      const int pg = ps_shift >= 0 ? slot >> ps_shift : slot / ps;
      const int page = free_pages[q.out_page_off + pg];
      if (page < 0 || page >= g.pool_pages) {
        if (lane == 0) report_error(status, CC_ERR_DEVICE_FLAG, 502);
        return;
      }
      dst0 = ((int64_t)page * ps + (slot - pg * ps)) * g.kv_stride_tok;
    }
    const int32_t* ip = idx + (int64_t)h0 * bt.b_tot + q.idx_off + slot;
#pragma unroll 1
    for (int hh = 0; hh < heads_per_group; hh += kUnroll) {
      int tok[kUnroll];
      int64_t src[kUnroll];
#pragma unroll
      for (int i = 0; i < kUnroll; ++i)
        tok[i] = hh + i < heads_per_group ? ip[(int64_t)(hh + i) * bt.b_tot] : INT_MIN;
#pragma unroll
      for (int i = 0; i < kUnroll; ++i) {
        src[i] = -1;
        if (tok[i] == INT_MIN) continue;                         // past the unit's last head
        if (tok[i] < 0 || tok[i] >= q.n) {
          if (lane == 0) report_error(status, CC_ERR_DEVICE_FLAG, 500);
          continue;
        }
        int64_t row;
        if (ps == 0) {
          row = (int64_t)q.tok_off + tok[i];
        } else {
          const int pg = ps_shift >= 0 ? tok[i] >> ps_shift : tok[i] / ps;
          const int page = pt[pg];
          if (page < 0 || page >= g.pool_pages) {
            if (lane == 0) report_error(status, CC_ERR_DEVICE_FLAG, 501);
            continue;
          }
          row = (int64_t)page * ps + (tok[i] - pg * ps);
        }
        src[i] = row * g.kv_stride_tok + (int64_t)(h0 + hh + i) * g.kv_stride_head;
      }
      uint4 kv[kUnroll], vv[kUnroll];
#pragma unroll
      for (int i = 0; i < kUnroll; ++i) {
        if (src[i] < 0) continue;
        kv[i] = ld_stream(reinterpret_cast<const uint4*>(k + src[i]) + lane);
        vv[i] = ld_stream(reinterpret_cast<const uint4*>(v + src[i]) + lane);
      }
#pragma unroll
      for (int i = 0; i < kUnroll; ++i) {
        if (src[i] < 0) continue;
        const int64_t dst = dst0 + (int64_t)(h0 + hh + i) * head_step;
        st_stream(reinterpret_cast<uint4*>(k_out + dst) + lane, kv[i]);
        st_stream(reinterpret_cast<uint4*>(v_out + dst) + lane, vv[i]);
      }
    }
  }
}

}  // namespace

cudaError_t launch_compact(const Launch& L, const BatchTable& bt, const Geometry& g,
                           const void* k, const void* v, const int32_t* idx, void* k_out,
                           void* v_out, const int32_t* free_pages, int32_t* out_page_table) {
  int64_t slots = 0;
  for (int s = 0; s < bt.num_seqs; ++s) slots += bt.seq[s].keep;
  // Heads per unit: all heads of a slot when the batch still fills the GPU that way (fewest
  // look-ups per byte), else one head per unit; the units of a slot must number a power of two.
  const int64_t full_wave = (int64_t)L.sm_count * 8 * kRowsPerBlock;
  int hpg = 1;
  if ((g.hkv & (g.hkv - 1)) != 0) {
    hpg = g.hkv;                                   // 1 unit per slot is the only power of two
  } else {
    for (int c = g.hkv; c > 1; c /= 2)
      if (slots * (g.hkv / c) >= full_wave) { hpg = c; break; }
  }
  int hc_shift = 0;
  while ((hpg << hc_shift) < g.hkv) ++hc_shift;
  int64_t blocks = 0;
  for (int s = 0; s < bt.num_seqs; ++s)
    blocks += max((int64_t)1, (((int64_t)bt.seq[s].keep << hc_shift) + kRowsPerBlock - 1) / kRowsPerBlock);
  dim3 grid((unsigned)blocks);
  auto kern = hpg >= 4 ? compact_kernel<4> : (hpg >= 2 ? compact_kernel<2> : compact_kernel<1>);
  return launch_pdl(kern, grid, dim3(kThreads), 0, L.stream, 1, bt, g, (const uint16_t*)k,
                    (const uint16_t*)v, idx, (uint16_t*)k_out, (uint16_t*)v_out, free_pages,
                    out_page_table, L.status, hpg, hc_shift);
}

}  // namespace cc
