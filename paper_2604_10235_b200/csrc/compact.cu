// A5: gather the retained K/V rows of every KV head into the compacted cache.
// Pure data movement: one 256-byte row of K and one of V per (slot, head), moved as
// 16-byte vectors by 16 consecutive threads, so every warp reads and writes two whole rows.
#include "cc_internal.cuh"

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

// grid: (blocks over slot*head pairs of the longest sequence, num_seqs)
__global__ void __launch_bounds__(kThreads, 8)      // 32 registers: eight blocks, all warp slots of an SM
compact_kernel(const __grid_constant__ BatchTable bt, const Geometry g,
               const uint16_t* __restrict__ k, const uint16_t* __restrict__ v,
               const int32_t* __restrict__ idx, uint16_t* __restrict__ k_out,
               uint16_t* __restrict__ v_out, const int32_t* __restrict__ free_pages,
               int32_t* __restrict__ out_page_table, DeviceStatus* status) {
  pdl_launch_dependents();
  pdl_wait();
  const int s = blockIdx.y;
  const SeqInfo& q = bt.seq[s];
  const int lane = threadIdx.x % kLanesPerRow;
  const int ps = bt.page_size;

  // the block with index 0 of each sequence also publishes the sequence's new page table
  if (ps > 0 && blockIdx.x == 0) {
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

  const int64_t pairs = (int64_t)q.keep * g.hkv;
  for (int64_t p = (int64_t)blockIdx.x * kRowsPerBlock + threadIdx.x / kLanesPerRow; p < pairs;
       p += (int64_t)gridDim.x * kRowsPerBlock) {
    const int slot = (int)(p / g.hkv);
    const int h = (int)(p % g.hkv);
    const int tok = idx[(int64_t)h * bt.b_tot + q.idx_off + slot];
    if (tok < 0 || tok >= q.n) {
      if (lane == 0) report_error(status, CC_ERR_DEVICE_FLAG, 500);
      continue;
    }
    const int64_t src_row = token_row(bt, g, s, tok);
    if (src_row < 0) {
      if (lane == 0) report_error(status, CC_ERR_DEVICE_FLAG, 501);
      continue;
    }
    int64_t dst;
    if (ps == 0) {
      dst = ((int64_t)q.idx_off + slot) * g.out_stride_tok + (int64_t)h * g.out_stride_head;
    } else {
      const int page = free_pages[q.out_page_off + slot / ps];
      if (page < 0 || page >= g.pool_pages) {
        if (lane == 0) report_error(status, CC_ERR_DEVICE_FLAG, 502);
        continue;
      }
      dst = ((int64_t)page * ps + slot % ps) * g.kv_stride_tok + (int64_t)h * g.kv_stride_head;
    }
    const int64_t src = src_row * g.kv_stride_tok + (int64_t)h * g.kv_stride_head;
    const uint4 kv = ld_stream(reinterpret_cast<const uint4*>(k + src) + lane);
    const uint4 vv = ld_stream(reinterpret_cast<const uint4*>(v + src) + lane);
    st_stream(reinterpret_cast<uint4*>(k_out + dst) + lane, kv);
    st_stream(reinterpret_cast<uint4*>(v_out + dst) + lane, vv);
  }
}

}  // namespace

cudaError_t launch_compact(const Launch& L, const BatchTable& bt, const Geometry& g,
                           const void* k, const void* v, const int32_t* idx, void* k_out,
                           void* v_out, const int32_t* free_pages, int32_t* out_page_table) {
  int max_keep = 0;
  for (int s = 0; s < bt.num_seqs; ++s) max_keep = max(max_keep, bt.seq[s].keep);
  int64_t pairs = (int64_t)max_keep * g.hkv;
  int blocks = (int)((pairs + kRowsPerBlock - 1) / kRowsPerBlock);
  if (blocks < 1) blocks = 1;
  const int cap = L.sm_count * 8;     // 8 resident blocks of 256 threads per SM
  if (blocks > cap) blocks = cap;
  dim3 grid(blocks, bt.num_seqs);
  return launch_pdl(compact_kernel, grid, dim3(kThreads), 0, L.stream, 1, bt, g, (const uint16_t*)k,
                    (const uint16_t*)v, idx, (uint16_t*)k_out, (uint16_t*)v_out, free_pages,
                    out_page_table, L.status);
}

}  // namespace cc
