// Materialising restore of one layer (Eq. 2; Sec. 4.2 "Cache restoration"):
//   restore_scale_kernel    x_hat = e_stored * (|x| / |e_stored|) for every cached row that was merged,
//                           then the retained rows from their raw copies (x_hat[I] = R)
#include <algorithm>

#include "mc_common.cuh"
#include "mc_items.cuh"
#include "mc_kernels.h"
#include "mc_pipe.cuh"

namespace mc {

constexpr int kRestoreThreads = 256;
constexpr int kRestoreWarps = kRestoreThreads / 32;
constexpr int kRestoreCtasPerSm = 2;
constexpr int kRowsPerItem = 64;
constexpr int kRestoreStages = 6;
// 64 rows of tiles: 64 / page_size whole (page, head) tiles, 16896 bytes for every page size
constexpr int kRestoreStageBytes = (kRowsPerItem / 16) * (16 * kRowBytes + 2 * 16 * 4);
constexpr int kRestoreAhead = kRestoreStages - 1;  // items in flight beyond the one being consumed

struct RestoreParams {
  Geom g;
  const char* e_pool[2];
  char* dst_pool[2];
  const int32_t* ret_count;
  const int32_t* ret_offset;
  const int32_t* ret_index;
  const char* ret_rows;
  int64_t ret_capacity;
  int layer;  // 0: l-1, 1: l
  int items_per_page;
  int32_t* status;
};

// Persistent: two CTAs per SM walk the items (64 rows of a page that holds tokens) with a fixed
// stride.  An item's tiles are one contiguous block of the pair cache; lane 0 of warp 0 streams
// them into a ring of shared-memory stages with one bulk asynchronous copy per item, five items
// ahead, so the bytes in flight are set by the ring.  A half-warp takes a row out of shared memory
// (undoing the chunk permutation), the stage is released as soon as the rows are in registers, and
// the scaled rows leave with streaming stores.
// F32: the dense rows are written as binary32 (the products e * scale unrounded, the raw rows of
// retained tokens converted exactly) instead of the 16-bit storage type.
template <int DT, bool F32>
__global__ void __launch_bounds__(kRestoreThreads, kRestoreCtasPerSm) restore_scale_kernel(const RestoreParams p) {
  constexpr int kOutRow = F32 ? 2 * kRowBytes : kRowBytes;  // bytes of a dense output row
  grid_dep_wait();
  grid_dep_launch();
  extern __shared__ unsigned char smem_raw[];
  unsigned char* smem = reinterpret_cast<unsigned char*>((reinterpret_cast<uintptr_t>(smem_raw) + 127) & ~uintptr_t(127));
  unsigned char* stages = smem;
  int* page_s = reinterpret_cast<int*>(smem + kRestoreStages * kRestoreStageBytes);  // [kRestoreStages]
  int* len_s = page_s + kRestoreStages;                                               // [batch]
  int* pre_s = len_s + kMaxBatchPages;                                                // [batch + 1]
  volatile int* s_abort = pre_s + kMaxBatchPages + 1;
  uint64_t* bars = reinterpret_cast<uint64_t*>((reinterpret_cast<uintptr_t>(s_abort + 1) + 7) & ~uintptr_t(7));
  const uint32_t full0 = smem_u32(bars), empty0 = full0 + 8 * kRestoreStages;
  const uint32_t stage0 = smem_u32(stages);
  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  const int ps = p.g.page_size, shift = p.g.page_shift, H = p.g.n_kv_heads;
  const int rows_in_page = H * ps;
  const int tbytes = tile_bytes(ps);

  if (tid == 0) {
    for (int s = 0; s < kRestoreStages; ++s) {
      mbar_init(full0 + 8 * s, 1);
      mbar_init(empty0 + 8 * s, kRestoreWarps);
    }
    *s_abort = 0;
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  page_prefix(p.g, len_s, pre_s, kRestoreThreads, p.status);
  const int P = pre_s[p.g.batch];
  const int ipp = p.items_per_page;
  const int stride = gridDim.x;
  const int s_pg = stride / ipp, s_grp = stride - s_pg * ipp;

  // a page id outside the pools comes back as -1: its item streams page 0 instead and writes nothing
  auto page_of = [&](const PageItem& m) { return m.tensor < 2 ? checked_page(p.g, m.b, m.pslot, p.status) : 0; };
  // lane 0 of warp 0: copy item j (the j-th item of this CTA) into stage j % kRestoreStages
  auto issue = [&](int j, const PageItem& m, int page_id) -> bool {
    const int page = max(page_id, 0);
    const int s = j % kRestoreStages;
    if (j >= kRestoreStages && !mbar_wait(empty0 + 8 * s, ((j / kRestoreStages) - 1) & 1, s_abort, p.status)) return false;
    const int h0 = (m.grp * kRowsPerItem) >> shift;
    const int n_tiles = min(kRowsPerItem >> shift, H - h0);
    const uint32_t bytes = (uint32_t)(n_tiles * tbytes);
    const uint32_t bar = full0 + 8 * s;
    page_s[s] = page_id;
    mbar_expect_tx(bar, bytes);
    bulk_load(stage0 + s * kRestoreStageBytes, (m.tensor ? p.e_pool[1] : p.e_pool[0]) + ((size_t)page * H + h0) * tbytes, bytes, bar);
    return true;
  };

  PageItem m;
  page_item_init(m, blockIdx.x, ipp, P, pre_s);
  // warp 0 keeps the issue point kRestoreAhead items ahead, and the page ids two items further (a
  // demand load takes microseconds while the copies saturate the memory system)
  PageItem mi = m, mn = m;
  int pg_i = 0, pg_n = 0;
  if (warp == 0) {
    pg_i = page_of(mi);
    page_item_advance(mn, s_pg, s_grp, ipp, P, pre_s);
    pg_n = page_of(mn);
#pragma unroll
    for (int j = 0; j < kRestoreAhead; ++j) {
      if (lane == 0 && mi.tensor < 2) issue(j, mi, pg_i);
      mi = mn;
      pg_i = pg_n;
      page_item_advance(mn, s_pg, s_grp, ipp, P, pre_s);
      pg_n = page_of(mn);
    }
  }

  const int hw = lane >> 4, l16 = lane & 15;
  for (int it = 0; m.tensor < 2; ++it) {
    if (warp == 0) {
      // item it + kRestoreAhead goes into the stage that item it - 1 has just left
      int good = 1;
      if (lane == 0 && mi.tensor < 2) good = issue(it + kRestoreAhead, mi, pg_i) ? 1 : 0;
      good = __shfl_sync(0xffffffffu, good, 0);
      if (!good) break;
      mi = mn;
      pg_i = pg_n;
      page_item_advance(mn, s_pg, s_grp, ipp, P, pre_s);
      pg_n = page_of(mn);
    }
    const int s = it % kRestoreStages;
    if (!mbar_wait(full0 + 8 * s, (it / kRestoreStages) & 1, s_abort, p.status)) break;
    const int page = page_s[s];
    const int n = len_s[m.b];
    // warp w: rows 8 w .. 8 w + 7 of the item, four per half-warp
    const int r0 = warp * 8 + hw * 4;
    const unsigned char* sb = stages + s * kRestoreStageBytes;
    uint4 v[4];
    float g[4];
    bool ok[4];
#pragma unroll
    for (int j = 0; j < 4; ++j) {
      const int r = r0 + j, rp = m.grp * kRowsPerItem + r;
      const int tk = r & (ps - 1);
      const unsigned char* tile = sb + (r >> shift) * tbytes;
      ok[j] = page >= 0 && rp < rows_in_page && m.pslot * ps + tk < n;
      v[j] = make_uint4(0u, 0u, 0u, 0u);
      g[j] = 0.f;
      if (ok[j]) {
        v[j] = *reinterpret_cast<const uint4*>(tile + tk * kRowBytes + chunk_pos(tk, l16) * 16);
        g[j] = reinterpret_cast<const float*>(tile + ps * kRowBytes)[p.layer * ps + tk];
      }
    }
    __syncwarp();
    if (lane == 0) mbar_arrive(empty0 + 8 * s);  // the stage is in registers now
#pragma unroll
    for (int j = 0; j < 4; ++j)  // a retained token (scale -0) is written from its raw row below, by whichever CTA gets there
      ok[j] = ok[j] && __float_as_uint(g[j]) != 0x80000000u;
    char* pd = (m.tensor ? p.dst_pool[1] : p.dst_pool[0]) +
               ((size_t)max(page, 0) * rows_in_page + m.grp * kRowsPerItem + r0) * kOutRow + l16 * (kOutRow / 16);
#pragma unroll
    for (int j = 0; j < 4; ++j)
      if (ok[j]) {
        const uint32_t w[4] = {v[j].x, v[j].y, v[j].z, v[j].w};
        uint32_t o[4];
        float2 f[4];
#pragma unroll
        for (int i = 0; i < 4; ++i) {
          f[i] = Elem<DT>::unpack(w[i]);
          f[i].x *= g[j];
          f[i].y *= g[j];
          o[i] = Elem<DT>::pack(f[i].x, f[i].y);
        }
        if (F32) {
          st_stream16(pd + j * kOutRow, make_uint4(__float_as_uint(f[0].x), __float_as_uint(f[0].y), __float_as_uint(f[1].x), __float_as_uint(f[1].y)));
          st_stream16(pd + j * kOutRow + 16, make_uint4(__float_as_uint(f[2].x), __float_as_uint(f[2].y), __float_as_uint(f[3].x), __float_as_uint(f[3].y)));
        } else {
          st_stream16(pd + j * kOutRow, make_uint4(o[0], o[1], o[2], o[3]));
        }
      }
    page_item_advance(m, s_pg, s_grp, ipp, P, pre_s);
  }
  // ---- x_hat[I] = R: the raw rows of the retained tokens, segments dealt round-robin to the CTAs,
  // a half-warp per row.  (The scaled rows above leave these tokens out, so the order is free.)
  {
    const int nseg = 2 * p.g.batch * H;
    const int hw16 = tid >> 4;
    for (int seg = blockIdx.x; seg < nseg; seg += gridDim.x) {
      const int cnt = p.ret_count[seg], off = p.ret_offset[seg];
      const int h = seg % H, b = (seg / H) % p.g.batch, tensor = seg / (H * p.g.batch);
      char* dst_pool = tensor ? p.dst_pool[1] : p.dst_pool[0];
      for (int e = hw16; e < cnt; e += kRestoreThreads / 16) {
        if (!MC_IN_BOUNDS(off >= 0 && (int64_t)off + e < p.ret_capacity, p.status)) continue;  // (range-checked build)
        const int tok = p.ret_index[off + e];
        if (!MC_IN_BOUNDS(tok >= 0 && tok < len_s[b], p.status)) continue;
        const int page = checked_page(p.g, b, tok >> shift, p.status);
        if (page < 0) continue;
        const size_t row = ((size_t)page * H + h) * ps + (tok & (ps - 1));
        const uint4 v = *reinterpret_cast<const uint4*>(p.ret_rows + ((size_t)p.layer * p.ret_capacity + off + e) * kRetEntryBytes +
                                                        l16 * 16);
        if (F32) {
          const float2 f0 = Elem<DT>::unpack(v.x), f1 = Elem<DT>::unpack(v.y), f2 = Elem<DT>::unpack(v.z), f3 = Elem<DT>::unpack(v.w);
          float4* d4 = reinterpret_cast<float4*>(dst_pool + row * kOutRow + l16 * 32);
          d4[0] = make_float4(f0.x, f0.y, f1.x, f1.y);
          d4[1] = make_float4(f2.x, f2.y, f3.x, f3.y);
        } else {
          *reinterpret_cast<uint4*>(dst_pool + row * kRowBytes + l16 * 16) = v;
        }
      }
    }
  }
  if (*s_abort) {
    for (int x = 0; x < 2000; ++x) __nanosleep(1000);  // let copies in flight land before the CTA's memory is released
  }
}

mc_status launch_restore(const mc_config* cfg, const mc_batch* bt, const Geom& g, const mc_pair_cache* pair,
                         int layer, const mc_layer_kv* dst, int dst_fp32, cudaStream_t stream) {
  if (bt->batch == 0) return MC_OK;
  RestoreParams rp;
  rp.g = g;
  rp.e_pool[0] = (const char*)pair->e_k;
  rp.e_pool[1] = (const char*)pair->e_v;
  rp.dst_pool[0] = (char*)dst->k_pool;
  rp.dst_pool[1] = (char*)dst->v_pool;
  rp.ret_count = pair->ret_count;
  rp.ret_offset = pair->ret_offset;
  rp.ret_index = pair->ret_index;
  rp.ret_rows = (const char*)pair->ret_rows;
  rp.ret_capacity = pair->ret_capacity;
  rp.layer = layer;
  rp.items_per_page = (cfg->n_kv_heads * cfg->page_size + kRowsPerItem - 1) / kRowsPerItem;
  rp.status = pair->status;
  if (bt->batch > kMaxBatchPages) return MC_ERR_SHAPE;  // the sequences' page prefix lives in shared memory
  // upper bound of the item count (the kernel enumerates the pages that hold tokens)
  const long long blocks = 2LL * bt->batch * ((bt->max_seq_len + cfg->page_size - 1) / cfg->page_size) * rp.items_per_page;
  if (blocks > 0x7fffffffLL) return MC_ERR_SHAPE;
  if (blocks > 0) {
    int n_sm = 0;
    if (mc_status st = sm_count(&n_sm)) return st;
    const int grid = (int)std::min<long long>((long long)n_sm * kRestoreCtasPerSm, blocks);
    const size_t smem = 128 + (size_t)kRestoreStages * kRestoreStageBytes + (kRestoreStages + 2 * kMaxBatchPages + 3) * 4 + 8 +
                        2 * kRestoreStages * 8 + 64;
    void (*kern)(const RestoreParams) =
        cfg->dtype == MC_F16 ? (dst_fp32 ? restore_scale_kernel<MC_F16, true> : restore_scale_kernel<MC_F16, false>)
                             : (dst_fp32 ? restore_scale_kernel<MC_BF16, true> : restore_scale_kernel<MC_BF16, false>);
    MC_CUDA_CHECK(cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem));
    MC_CUDA_CHECK(launch_pdl(kern, dim3(grid), dim3(kRestoreThreads), smem, stream, rp));
    MC_CUDA_CHECK(cudaGetLastError());
  }
  return MC_OK;
}

}  // namespace mc
