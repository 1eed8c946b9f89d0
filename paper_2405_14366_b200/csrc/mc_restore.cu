// Materialising restore of one layer (Eq. 2; Sec. 4.2 "Cache restoration"):
//   restore_scale_kernel    x_hat = e_stored * (|x| / |e_stored|) for every cached row
//   restore_scatter_kernel  retained rows overwritten with their raw copies (x_hat[I] = R)
#include "mc_common.cuh"
#include "mc_kernels.h"

namespace mc {

constexpr int kRestoreThreads = 256;
constexpr int kRowsPerItem = 64;
constexpr int kRowsPerHalfWarp = 4;

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
};

template <int DT>
__global__ void __launch_bounds__(kRestoreThreads) restore_scale_kernel(const RestoreParams p) {
  grid_dep_wait();
  grid_dep_launch();
  const int ipp = p.items_per_page;
  int bid = blockIdx.x;
  const int item = bid % ipp;
  bid /= ipp;
  const int pslot = bid % p.g.max_pages_per_seq;
  bid /= p.g.max_pages_per_seq;
  const int b = bid % p.g.batch;
  const int tensor = bid / p.g.batch;
  const int n = p.g.seq_lens[b];
  const int ps = p.g.page_size;
  if (pslot * ps >= n) return;
  const int page = p.g.block_table[(size_t)b * p.g.max_pages_per_seq + pslot];
  const int H = p.g.n_kv_heads;
  const int rows_in_page = H * ps;
  const int hw = threadIdx.x >> 4, l16 = threadIdx.x & 15;
  const int row0 = item * kRowsPerItem + hw * kRowsPerHalfWarp;
  if (row0 >= rows_in_page) return;
  const int head = row0 >> p.g.page_shift;
  const int tk0 = row0 & (ps - 1);
  const int tok0 = pslot * ps + tk0;
  const size_t page_off = (size_t)page * rows_in_page;
  const char* tile = p.e_pool[tensor] + ((size_t)page * H + head) * tile_bytes(ps);
  char* pd = p.dst_pool[tensor] + (page_off + row0) * kRowBytes + l16 * 16;
  const float* sc = reinterpret_cast<const float*>(tile + ps * kRowBytes) + p.layer * ps + tk0;
  uint4 v[kRowsPerHalfWarp];
  float g[kRowsPerHalfWarp];
#pragma unroll
  for (int j = 0; j < kRowsPerHalfWarp; ++j)
    if (tok0 + j < n) {
      v[j] = ld_stream16(tile + (tk0 + j) * kRowBytes + chunk_pos(tk0 + j, l16) * 16);
      g[j] = __ldg(sc + j);
    }
#pragma unroll
  for (int j = 0; j < kRowsPerHalfWarp; ++j)
    if (tok0 + j < n) {
      const uint32_t w[4] = {v[j].x, v[j].y, v[j].z, v[j].w};
      uint32_t o[4];
#pragma unroll
      for (int i = 0; i < 4; ++i) {
        const float2 f = Elem<DT>::unpack(w[i]);
        o[i] = Elem<DT>::pack(f.x * g[j], f.y * g[j]);
      }
      st_stream16(pd + j * kRowBytes, make_uint4(o[0], o[1], o[2], o[3]));
    }
}

__global__ void __launch_bounds__(kRestoreThreads) restore_scatter_kernel(const RestoreParams p) {
  grid_dep_wait();
  grid_dep_launch();
  const int seg = blockIdx.y;
  const int H = p.g.n_kv_heads;
  const int h = seg % H;
  const int b = (seg / H) % p.g.batch;
  const int tensor = seg / (H * p.g.batch);
  const int cnt = p.ret_count[seg];
  const int off = p.ret_offset[seg];
  const int hw = threadIdx.x >> 4, l16 = threadIdx.x & 15;
  for (int e = blockIdx.x * (kRestoreThreads / 16) + hw; e < cnt; e += gridDim.x * (kRestoreThreads / 16)) {
    const int tok = p.ret_index[off + e];
    const int page = p.g.block_table[(size_t)b * p.g.max_pages_per_seq + (tok >> p.g.page_shift)];
    const size_t row = ((size_t)page * H + h) * p.g.page_size + (tok & (p.g.page_size - 1));
    const uint4 v =
        *reinterpret_cast<const uint4*>(p.ret_rows + ((size_t)p.layer * p.ret_capacity + off + e) * kRetEntryBytes + l16 * 16);
    *reinterpret_cast<uint4*>(p.dst_pool[tensor] + row * kRowBytes + l16 * 16) = v;
  }
}

mc_status launch_restore(const mc_config* cfg, const mc_batch* bt, const Geom& g, const mc_pair_cache* pair,
                         int layer, const mc_layer_kv* dst, cudaStream_t stream) {
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
  const long long blocks = 2LL * bt->batch * bt->max_pages_per_seq * rp.items_per_page;
  if (blocks > 0x7fffffffLL) return MC_ERR_SHAPE;
  if (blocks > 0) {
    if (cfg->dtype == MC_F16)
      MC_CUDA_CHECK(launch_pdl(restore_scale_kernel<MC_F16>, dim3((unsigned)blocks), dim3(kRestoreThreads), 0, stream, rp));
    else
      MC_CUDA_CHECK(launch_pdl(restore_scale_kernel<MC_BF16>, dim3((unsigned)blocks), dim3(kRestoreThreads), 0, stream, rp));
    MC_CUDA_CHECK(cudaGetLastError());
  }
  const int nseg = 2 * bt->batch * cfg->n_kv_heads;
  dim3 grid(4, nseg);
  MC_CUDA_CHECK(launch_pdl(restore_scatter_kernel, dim3(grid), dim3(kRestoreThreads), 0, stream, rp));
  MC_CUDA_CHECK(cudaGetLastError());
  return MC_OK;
}

}  // namespace mc
