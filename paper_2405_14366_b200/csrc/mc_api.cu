// C-ABI entry points: argument validation and dispatch to the kernel launchers.
#include <stdio.h>
#include <string.h>

#include <atomic>
#include <vector>

#include <nvtx3/nvToolsExt.h>

#include "mc_common.cuh"
#include "mc_items.cuh"
#include "mc_kernels.h"
#include "mc_append.cuh"
#include "mc_q4.cuh"

namespace mc {

static thread_local char g_cuda_error[256] = "";

void set_cuda_error(cudaError_t e, const char* where) {
  snprintf(g_cuda_error, sizeof(g_cuda_error), "%s: %s", where, cudaGetErrorString(e));
  (void)cudaGetLastError();  // clear the sticky-free error state
}

mc_status sm_count(int* n_sm) {
  constexpr int kMaxDev = 64;
  static std::atomic<int> cache[kMaxDev];  // zero-initialised; 0 = not looked up yet
  int dev = 0;
  MC_CUDA_CHECK(cudaGetDevice(&dev));
  int v = (dev >= 0 && dev < kMaxDev) ? cache[dev].load(std::memory_order_relaxed) : 0;
  if (v == 0) {
    MC_CUDA_CHECK(cudaDeviceGetAttribute(&v, cudaDevAttrMultiProcessorCount, dev));
    if (dev >= 0 && dev < kMaxDev) cache[dev].store(v, std::memory_order_relaxed);
  }
  *n_sm = v;
  return MC_OK;
}

// A named range around every compute entry point: visible on a profiler's timeline, a no-op (one
// indirect call) when no tool is attached.
struct ApiRange {
  explicit ApiRange(const char* name) { nvtxRangePushA(name); }
  ~ApiRange() { nvtxRangePop(); }
};

static bool aligned256(const void* p) { return (reinterpret_cast<uintptr_t>(p) & 255u) == 0; }

static mc_status check_config(const mc_config* cfg) {
  if (cfg == nullptr) return MC_ERR_INVALID_ARG;
  if (cfg->head_dim != kHeadDim) return MC_ERR_SHAPE;
  if (cfg->page_size != 16 && cfg->page_size != 32 && cfg->page_size != 64) return MC_ERR_SHAPE;
  if (cfg->n_kv_heads <= 0 || cfg->n_q_heads <= 0 || cfg->n_q_heads % cfg->n_kv_heads != 0) return MC_ERR_SHAPE;
  const int nq = cfg->n_q_heads / cfg->n_kv_heads;
  if (nq != 1 && nq != 2 && nq != 4 && nq != 8) return MC_ERR_SHAPE;
  if (cfg->dtype != MC_F16 && cfg->dtype != MC_BF16) return MC_ERR_DTYPE;
  if (cfg->retain_mode < MC_RETAIN_DISTINCT || cfg->retain_mode > MC_RETAIN_TOPK) return MC_ERR_INVALID_ARG;
  if (cfg->merge_fn < MC_MERGE_SLERP || cfg->merge_fn > MC_MERGE_MEAN) return MC_ERR_INVALID_ARG;
  if (cfg->cache_bits != 0 && cfg->cache_bits != 16 && cfg->cache_bits != 4) return MC_ERR_INVALID_ARG;
  if (cfg->cache_bits == 4 && cfg->page_size != kQ4Page) return MC_ERR_SHAPE;
  if (cfg->t_mode != MC_T_FIXED && cfg->t_mode != MC_T_MAGNITUDE_RATIO) return MC_ERR_INVALID_ARG;
  if (cfg->retain_union != 0 && cfg->retain_union != 1) return MC_ERR_INVALID_ARG;
  if (cfg->retain_union && cfg->retain_mode == MC_RETAIN_TOPK) return MC_ERR_UNSUPPORTED;
  if (cfg->append_slack < 0 || cfg->append_slack > 65536) return MC_ERR_INVALID_ARG;
  if (!(cfg->t >= 0.0 && cfg->t <= 1.0) || !(cfg->gamma >= 0.0 && cfg->gamma <= 1.0)) return MC_ERR_INVALID_ARG;
  return MC_OK;
}

static mc_status check_batch(const mc_config* cfg, const mc_batch* bt) {
  if (bt == nullptr) return MC_ERR_INVALID_ARG;
  if (bt->batch < 0 || bt->max_pages_per_seq < 0 || bt->max_seq_len < 0 || bt->n_pages < 0) return MC_ERR_INVALID_ARG;
  if (bt->batch > 0 && (bt->block_table == nullptr || bt->seq_lens == nullptr)) return MC_ERR_INVALID_ARG;
  if ((long long)bt->max_pages_per_seq * cfg->page_size < bt->max_seq_len) return MC_ERR_SHAPE;
  if (2LL * bt->batch * cfg->n_kv_heads > 65535) return MC_ERR_SHAPE;  // one grid row per segment
  if (bt->n_pages * cfg->n_kv_heads * cfg->page_size > 0x7fffffffLL) return MC_ERR_SHAPE;
  return MC_OK;
}

static mc_status check_pair(const mc_config* cfg, const mc_pair_cache* pc) {
  if (pc == nullptr) return MC_ERR_INVALID_ARG;
  if (cfg->cache_bits == 4) {
    if (!pc->res_k || !pc->res_v) return MC_ERR_INVALID_ARG;
    if (!aligned256(pc->res_k) || !aligned256(pc->res_v)) return MC_ERR_ALIGN;
  }
  if (!pc->e_k || !pc->e_v || !pc->dist || !pc->ret_count || !pc->ret_offset || !pc->seg_minmax ||
      !pc->status)
    return MC_ERR_INVALID_ARG;
  if (pc->ret_capacity < 0 || pc->ret_prefix == nullptr || pc->ret_prefix_stride < 2) return MC_ERR_INVALID_ARG;
  if (pc->ret_capacity > 0 && (!pc->ret_index || !pc->ret_rows)) return MC_ERR_INVALID_ARG;
  if (!aligned256(pc->e_k) || !aligned256(pc->e_v) || !aligned256(pc->dist)) return MC_ERR_ALIGN;
  if (pc->ret_rows && !aligned256(pc->ret_rows)) return MC_ERR_ALIGN;
  return MC_OK;
}

static Geom make_geom(const mc_config* cfg, const mc_batch* bt) {
  Geom g;
  g.block_table = bt->block_table;
  g.seq_lens = bt->seq_lens;
  g.batch = bt->batch;
  g.max_pages_per_seq = bt->max_pages_per_seq;
  g.n_kv_heads = cfg->n_kv_heads;
  g.page_size = cfg->page_size;
  g.page_shift = cfg->page_size == 16 ? 4 : (cfg->page_size == 32 ? 5 : 6);
  g.max_seq_len = bt->max_seq_len;
  g.n_pages = (int)bt->n_pages;
  g.seq_begin = 0;
  g.seq_count = bt->batch;
  return g;
}

// Merge scratch: the retention tables, and for the 4-bit shared cache the 16-bit staging tiles of both tensors.
static size_t merge_workspace_total(const mc_config* cfg, const mc_batch* bt) {
  return merge_workspace_bytes(cfg, bt) + (cfg->cache_bits == 4 ? 2 * q4_stage_bytes(cfg, bt) : 0);
}

// Runs the merge; with a 4-bit shared cache the kernels write 16-bit tiles into the staging part of the
// workspace (retention marks its tokens there), which then become 4-bit tiles and residual tiles.
static mc_status run_merge(const mc_config* cfg, const mc_batch* batch, const mc_layer_kv* lm1, const mc_layer_kv* l,
                           const mc_layer_q4* q_lm1, const mc_layer_q4* q_l, const mc_pair_cache* out, int do_retention,
                           void* workspace, cudaStream_t stream) {
  const Geom g = make_geom(cfg, batch);
  if (cfg->cache_bits != 4) return launch_merge(cfg, batch, g, lm1, l, q_lm1, q_l, out, do_retention, workspace, stream);
  mc_pair_cache stg = *out;
  char* base = (char*)workspace + merge_workspace_bytes(cfg, batch);
  stg.e_k = base;
  stg.e_v = base + q4_stage_bytes(cfg, batch);
  mc_status st = launch_merge(cfg, batch, g, lm1, l, q_lm1, q_l, &stg, do_retention, workspace, stream);
  if (st != MC_OK) return st;
  return launch_q4_quantise(cfg, batch, g, stg.e_k, stg.e_v, out, stream);
}

}  // namespace mc

using namespace mc;

extern "C" {

int32_t mc_version(void) { return 240; }

int32_t mc_build_flags(void) {
#if defined(MC_BOUNDS) && MC_BOUNDS
  return MC_BUILD_BOUNDS;
#else
  return 0;
#endif
}

const char* mc_status_str(int32_t s) {
  switch (s) {
    case MC_OK: return "MC_OK";
    case MC_ERR_INVALID_ARG: return "MC_ERR_INVALID_ARG";
    case MC_ERR_SHAPE: return "MC_ERR_SHAPE";
    case MC_ERR_DTYPE: return "MC_ERR_DTYPE";
    case MC_ERR_ALIGN: return "MC_ERR_ALIGN";
    case MC_ERR_CAPACITY: return "MC_ERR_CAPACITY";
    case MC_ERR_UNSUPPORTED: return "MC_ERR_UNSUPPORTED";
    case MC_ERR_CUDA: return "MC_ERR_CUDA";
    case MC_ERR_DEVICE_STATUS: return "MC_ERR_DEVICE_STATUS";
    default: return "MC_ERR_UNKNOWN";
  }
}

const char* mc_last_cuda_error(void) { return g_cuda_error; }

mc_status mc_workspace_bytes(const mc_config* cfg, const mc_batch* batch, int32_t op, int32_t n_query_sets,
                             size_t* bytes) {
  mc_status st = check_config(cfg);
  if (st != MC_OK) return st;
  if (batch == nullptr || bytes == nullptr) return MC_ERR_INVALID_ARG;
  if (batch->batch < 0 || batch->max_seq_len < 0) return MC_ERR_INVALID_ARG;
  if (op == MC_OP_MERGE) {
    if (batch->n_pages < 0) return MC_ERR_INVALID_ARG;
    *bytes = merge_workspace_total(cfg, batch) + 256;
  } else if (op == MC_OP_DECODE_ATTN) {
    if (n_query_sets != 1 && n_query_sets != 2) return MC_ERR_INVALID_ARG;
    *bytes = attn_workspace_bytes(cfg, batch, n_query_sets) + 256;
  } else {
    return MC_ERR_INVALID_ARG;
  }
  return MC_OK;
}

// What every form of the merge call checks about the output pair and the scratch memory.
static mc_status check_merge_common(const mc_config* cfg, const mc_batch* batch, const mc_pair_cache* out, void* workspace,
                                    size_t workspace_bytes) {
  mc_status st = check_pair(cfg, out);
  if (st != MC_OK) return st;
  if (batch->batch > kMaxBatchPages) return MC_ERR_SHAPE;  // the sequences' page prefix lives in shared memory
  if (workspace == nullptr || !aligned256(workspace)) return workspace ? MC_ERR_ALIGN : MC_ERR_INVALID_ARG;
  if (workspace_bytes < merge_workspace_total(cfg, batch)) return MC_ERR_CAPACITY;
  if (out->ret_prefix_stride < (batch->max_seq_len + 127) / 128 + 1) return MC_ERR_CAPACITY;
  return MC_OK;
}

mc_status mc_pair_bytes(const mc_config* cfg, const mc_batch* batch, int64_t ret_capacity, mc_pair_sizes* out) {
  mc_status st = check_config(cfg);
  if (st != MC_OK) return st;
  if (batch == nullptr || out == nullptr) return MC_ERR_INVALID_ARG;
  if (batch->batch < 0 || batch->max_seq_len < 0 || batch->n_pages < 0 || ret_capacity < 0) return MC_ERR_INVALID_ARG;
  const size_t nseg = (size_t)2 * batch->batch * cfg->n_kv_heads;
  const size_t ph = (size_t)batch->n_pages * cfg->n_kv_heads;
  memset(out, 0, sizeof(*out));
  const bool q4 = cfg->cache_bits == 4;
  out->tile_bytes = q4 ? (size_t)kQ4TileBytes : (size_t)tile_bytes(cfg->page_size);
  out->e_bytes = ph * out->tile_bytes;
  out->res_bytes = q4 ? (size_t)batch->batch * cfg->n_kv_heads * kResTileBytes : 0;
  out->dist_bytes = ph * 2 * cfg->page_size * sizeof(float);
  out->ret_count_bytes = nseg * sizeof(int32_t);
  out->ret_offset_bytes = (nseg + 1) * sizeof(int32_t);
  out->ret_index_bytes = (size_t)ret_capacity * sizeof(int32_t);
  out->ret_rows_bytes = (size_t)2 * ret_capacity * kRetEntryBytes;
  out->ret_prefix_stride = (batch->max_seq_len + 127) / 128 + 1;
  out->ret_prefix_bytes = nseg * (size_t)out->ret_prefix_stride * sizeof(int32_t);
  out->seg_minmax_bytes = nseg * 2 * sizeof(float);
  out->status_bytes = MC_STATUS_WORDS * sizeof(int32_t);
  const size_t parts[] = {out->e_bytes, out->e_bytes, out->dist_bytes, out->ret_count_bytes, out->ret_offset_bytes,
                          out->ret_index_bytes, out->ret_rows_bytes, out->ret_prefix_bytes, out->seg_minmax_bytes,
                          out->status_bytes, out->res_bytes, out->res_bytes};
  for (size_t b : parts) out->total_bytes += align_up(b, 256);
  return MC_OK;
}

mc_status mc_get_stats(const mc_config* cfg, const mc_batch* batch, const mc_pair_cache* pair, void* stream,
                       mc_stats* out) {
  ApiRange range_("mc_get_stats");
  mc_status st = check_config(cfg);
  if (st != MC_OK) return st;
  st = check_batch(cfg, batch);
  if (st != MC_OK) return st;
  if (pair == nullptr || pair->status == nullptr || out == nullptr) return MC_ERR_INVALID_ARG;
  memset(out, 0, sizeof(*out));
  cudaStream_t s = (cudaStream_t)stream;
  int32_t words[MC_STATUS_WORDS];
  std::vector<int32_t> lens_v((size_t)batch->batch + 1);
  int32_t* lens = lens_v.data();
  MC_CUDA_CHECK(cudaMemcpyAsync(words, pair->status, sizeof(words), cudaMemcpyDeviceToHost, s));
  if (batch->batch > 0)
    MC_CUDA_CHECK(cudaMemcpyAsync(lens, batch->seq_lens, (size_t)batch->batch * sizeof(int32_t), cudaMemcpyDeviceToHost, s));
  MC_CUDA_CHECK(cudaStreamSynchronize(s));
  int64_t tokens = 0, pages = 0, tokens_q = 0;
  for (int b = 0; b < batch->batch; ++b) {
    const int64_t n = lens[b] < 0 ? 0 : lens[b];
    tokens += n;
    pages += (n + cfg->page_size - 1) / cfg->page_size;
    tokens_q += n / kQ4Page * kQ4Page;  // tokens in complete pages
  }
  const int64_t th = tokens * cfg->n_kv_heads;  // (token, kv head) rows per layer and tensor
  out->flags = words[MC_STATUS_FLAGS];
  out->retained_total = words[MC_STATUS_RETAINED_TOTAL];
  out->near_threshold = words[MC_STATUS_NEAR_THRESHOLD];
  out->token_heads = th;
  out->full_bytes = 2 * 2 * th * kRowBytes;  // two layers, K and V
  // the shared direction row, both magnitudes and the distance per (token, head, tensor); both raw rows
  // and the index per retained entry
  out->compressed_bytes = 2 * th * (kRowBytes + 3 * 4) + out->retained_total * (2 * kRowBytes + 4);
  if (cfg->cache_bits == 4) {
    // a row in a complete page: 64 bytes of codes and its share of the group parameters (keys: 128 x 4
    // bytes per 32 tokens, values: 4 x 4 bytes per token: 16 either way); the residual rows stay 16-bit
    const int64_t thq = tokens_q * cfg->n_kv_heads;
    out->compressed_bytes = 2 * thq * (64 + 16 + 3 * 4) + 2 * (th - thq) * (kRowBytes + 3 * 4) +
                            out->retained_total * (2 * kRowBytes + 4);
  }
  // what the pair occupies in the caller's buffers: whole tiles of the pages in use, the distances, the
  // padded retained entries, the per-segment tables
  const int64_t nseg = 2LL * batch->batch * cfg->n_kv_heads;
  const int64_t tile_b = cfg->cache_bits == 4 ? kQ4TileBytes : tile_bytes(cfg->page_size);
  const int64_t res_b = cfg->cache_bits == 4 ? 2LL * batch->batch * cfg->n_kv_heads * kResTileBytes : 0;
  out->stored_bytes = res_b + 2 * pages * cfg->n_kv_heads * (tile_b + cfg->page_size * 4) +
                      out->retained_total * (2 * kRetEntryBytes + 4) +
                      nseg * (4 + 4 + 8 + 4 * pair->ret_prefix_stride) + 4 + MC_STATUS_WORDS * 4;
  if (out->flags & MC_FLAG_RETAIN_OVERFLOW) return MC_ERR_CAPACITY;
  if (out->flags != 0) return MC_ERR_DEVICE_STATUS;
  return MC_OK;
}

mc_status mc_merge_pair(const mc_config* cfg, const mc_batch* batch, const mc_layer_kv* lm1, const mc_layer_kv* l,
                        const mc_pair_cache* out, int32_t do_retention, void* workspace, size_t workspace_bytes,
                        void* stream) {
  ApiRange range_("mc_merge_pair");
  mc_status st = check_config(cfg);
  if (st != MC_OK) return st;
  st = check_batch(cfg, batch);
  if (st != MC_OK) return st;
  if (!lm1 || !l || !lm1->k_pool || !lm1->v_pool || !l->k_pool || !l->v_pool) return MC_ERR_INVALID_ARG;
  if (!aligned256(lm1->k_pool) || !aligned256(lm1->v_pool) || !aligned256(l->k_pool) || !aligned256(l->v_pool))
    return MC_ERR_ALIGN;
  st = check_merge_common(cfg, batch, out, workspace, workspace_bytes);
  if (st != MC_OK) return st;
  return run_merge(cfg, batch, lm1, l, nullptr, nullptr, out, do_retention ? 1 : 0, workspace, (cudaStream_t)stream);
}

mc_status mc_merge_pairs(const mc_config* cfg, const mc_batch* batch, int32_t n_pairs, const mc_layer_kv* const* lm1,
                         const mc_layer_kv* const* l, const mc_pair_cache* const* out, int32_t do_retention, void* workspace,
                         size_t workspace_bytes, void* stream) {
  ApiRange range_("mc_merge_pairs");
  mc_status st = check_config(cfg);
  if (st != MC_OK) return st;
  st = check_batch(cfg, batch);
  if (st != MC_OK) return st;
  if (n_pairs < 0 || !lm1 || !l || !out) return MC_ERR_INVALID_ARG;
  if (cfg->cache_bits == 4) return MC_ERR_UNSUPPORTED;  // the 4-bit cache is merged pair by pair (mc_merge_pair)
  if (workspace == nullptr || !aligned256(workspace)) return workspace ? MC_ERR_ALIGN : MC_ERR_INVALID_ARG;
  const size_t ws_pair = merge_workspace_bytes(cfg, batch);
  if (workspace_bytes < (size_t)n_pairs * ws_pair) return MC_ERR_CAPACITY;
  // every pair is checked before anything is launched
  for (int i = 0; i < n_pairs; ++i) {
    if (!lm1[i] || !l[i] || !lm1[i]->k_pool || !lm1[i]->v_pool || !l[i]->k_pool || !l[i]->v_pool) return MC_ERR_INVALID_ARG;
    if (!aligned256(lm1[i]->k_pool) || !aligned256(lm1[i]->v_pool) || !aligned256(l[i]->k_pool) || !aligned256(l[i]->v_pool))
      return MC_ERR_ALIGN;
    st = check_merge_common(cfg, batch, out[i], workspace, ws_pair);
    if (st != MC_OK) return st;
    for (int j = 0; j < i; ++j)
      if (out[j] == out[i] || out[j]->status == out[i]->status) return MC_ERR_INVALID_ARG;  // one pair cache per pair
  }
  const Geom g = make_geom(cfg, batch);
  for (int i0 = 0; i0 < n_pairs; i0 += kMergePairsPerLaunch) {
    const int n = n_pairs - i0 < kMergePairsPerLaunch ? n_pairs - i0 : kMergePairsPerLaunch;
    st = launch_merge_pairs(cfg, batch, g, n, lm1 + i0, l + i0, nullptr, nullptr, out + i0, do_retention ? 1 : 0,
                            (char*)workspace + (size_t)i0 * ws_pair, (cudaStream_t)stream);
    if (st != MC_OK) return st;
  }
  return MC_OK;
}

mc_status mc_admit_sequences(const mc_config* cfg, const mc_batch* batch, int32_t seq_begin, int32_t seq_count, int32_t n_pairs,
                             const mc_layer_kv* const* lm1, const mc_layer_kv* const* l, const mc_layer_q4* const* q4_lm1,
                             const mc_layer_q4* const* q4_l, const mc_pair_cache* const* out, int64_t rows_per_seq,
                             int32_t do_retention, void* workspace, size_t workspace_bytes, void* stream) {
  ApiRange range_("mc_admit_sequences");
  mc_status st = check_config(cfg);
  if (st != MC_OK) return st;
  st = check_batch(cfg, batch);
  if (st != MC_OK) return st;
  const bool q4 = q4_lm1 != nullptr;
  if (n_pairs < 0 || !out || (q4 ? (!q4_l || lm1 || l) : (!lm1 || !l || q4_l))) return MC_ERR_INVALID_ARG;
  if (seq_begin < 0 || seq_count < 0 || seq_begin + (int64_t)seq_count > batch->batch) return MC_ERR_INVALID_ARG;
  if (rows_per_seq <= 0 || rows_per_seq > 0x7fffffff / (batch->batch > 0 ? batch->batch : 1)) return MC_ERR_INVALID_ARG;
  if (q4 && cfg->page_size != kQ4Page) return MC_ERR_SHAPE;
  if (workspace == nullptr || !aligned256(workspace)) return workspace ? MC_ERR_ALIGN : MC_ERR_INVALID_ARG;
  const size_t ws_pair = merge_workspace_bytes(cfg, batch);
  const size_t ws_stage = cfg->cache_bits == 4 ? 2 * q4_stage_bytes(cfg, batch) : 0;
  if (workspace_bytes < (size_t)n_pairs * ws_pair + ws_stage) return MC_ERR_CAPACITY;
  for (int i = 0; i < n_pairs; ++i) {
    const void* ptrs[8];
    if (q4) {
      if (!q4_lm1[i] || !q4_l[i]) return MC_ERR_INVALID_ARG;
      const void* pp[8] = {q4_lm1[i]->k_codes, q4_lm1[i]->k_meta, q4_lm1[i]->v_codes, q4_lm1[i]->v_meta,
                           q4_l[i]->k_codes,   q4_l[i]->k_meta,   q4_l[i]->v_codes,   q4_l[i]->v_meta};
      memcpy(ptrs, pp, sizeof(pp));
    } else {
      if (!lm1[i] || !l[i]) return MC_ERR_INVALID_ARG;
      const void* pp[8] = {lm1[i]->k_pool, lm1[i]->v_pool, l[i]->k_pool, l[i]->v_pool, lm1[i]->k_pool, lm1[i]->v_pool, l[i]->k_pool, l[i]->v_pool};
      memcpy(ptrs, pp, sizeof(pp));
    }
    for (const void* q : ptrs) {
      if (q == nullptr) return MC_ERR_INVALID_ARG;
      if (!aligned256(q)) return MC_ERR_ALIGN;
    }
    st = check_merge_common(cfg, batch, out[i], workspace, ws_pair + ws_stage);
    if (st != MC_OK) return st;
    if ((int64_t)batch->batch * rows_per_seq > out[i]->ret_capacity) return MC_ERR_CAPACITY;
    for (int j = 0; j < i; ++j)
      if (out[j] == out[i] || out[j]->status == out[i]->status) return MC_ERR_INVALID_ARG;
  }
  Geom g = make_geom(cfg, batch);
  g.seq_begin = seq_begin;
  g.seq_count = seq_count;
  cudaStream_t s = (cudaStream_t)stream;
  if (cfg->cache_bits == 4) {
    // one pair after the other through the one staging area: merge into 16-bit tiles, then quantise
    char* stage = (char*)workspace + (size_t)n_pairs * ws_pair;
    for (int i = 0; i < n_pairs; ++i) {
      mc_pair_cache stg = *out[i];
      stg.e_k = stage;
      stg.e_v = stage + q4_stage_bytes(cfg, batch);
      const mc_pair_cache* sp = &stg;
      st = launch_merge_pairs(cfg, batch, g, 1, q4 ? nullptr : lm1 + i, q4 ? nullptr : l + i, q4 ? q4_lm1 + i : nullptr,
                              q4 ? q4_l + i : nullptr, &sp, do_retention ? 1 : 0, (char*)workspace + (size_t)i * ws_pair, s,
                              (int)rows_per_seq);
      if (st != MC_OK) return st;
      st = launch_q4_quantise(cfg, batch, g, stg.e_k, stg.e_v, out[i], s);
      if (st != MC_OK) return st;
    }
    return MC_OK;
  }
  for (int i0 = 0; i0 < n_pairs; i0 += kMergePairsPerLaunch) {
    const int n = n_pairs - i0 < kMergePairsPerLaunch ? n_pairs - i0 : kMergePairsPerLaunch;
    st = launch_merge_pairs(cfg, batch, g, n, q4 ? nullptr : lm1 + i0, q4 ? nullptr : l + i0, q4 ? q4_lm1 + i0 : nullptr,
                            q4 ? q4_l + i0 : nullptr, out + i0, do_retention ? 1 : 0, (char*)workspace + (size_t)i0 * ws_pair, s,
                            (int)rows_per_seq);
    if (st != MC_OK) return st;
  }
  return MC_OK;
}

mc_status mc_prefill_merge_pair(const mc_config* cfg, const mc_batch* batch, const mc_projection* proj, const mc_layer_kv* lm1,
                                const mc_layer_kv* l, const mc_pair_cache* out, float d_hint, int32_t do_retention,
                                void* workspace, size_t workspace_bytes, void* stream) {
  ApiRange range_("mc_prefill_merge_pair");
  mc_status st = check_config(cfg);
  if (st != MC_OK) return st;
  st = check_batch(cfg, batch);
  if (st != MC_OK) return st;
  if (!proj || !proj->x || !proj->w_k || !proj->w_v || !lm1 || !l || !lm1->k_pool || !lm1->v_pool || !l->k_pool || !l->v_pool)
    return MC_ERR_INVALID_ARG;
  if (proj->d_model <= 0 || proj->d_model % 64 != 0 || proj->x_seq_stride <= 0 || proj->x_seq_stride % 128 != 0 ||
      proj->x_seq_stride < batch->max_seq_len)
    return MC_ERR_SHAPE;
  if (cfg->merge_fn != MC_MERGE_SLERP || cfg->cache_bits == 4) return MC_ERR_UNSUPPORTED;
  if (do_retention && cfg->retain_mode != MC_RETAIN_DISTINCT && d_hint >= 0.f) return MC_ERR_UNSUPPORTED;
  if (do_retention && cfg->retain_union && d_hint >= 0.f) return MC_ERR_UNSUPPORTED;  // the other tensor's rule may keep a token below the hint
  if (!aligned256(proj->x) || !aligned256(proj->w_k) || !aligned256(proj->w_v) || !aligned256(lm1->k_pool) ||
      !aligned256(lm1->v_pool) || !aligned256(l->k_pool) || !aligned256(l->v_pool))
    return MC_ERR_ALIGN;
  st = check_merge_common(cfg, batch, out, workspace, workspace_bytes);
  if (st != MC_OK) return st;
  PrefillHook hook = {proj, d_hint};
  return launch_merge_pairs(cfg, batch, make_geom(cfg, batch), 1, &lm1, &l, nullptr, nullptr, &out, do_retention ? 1 : 0, workspace,
                            (cudaStream_t)stream, 0, &hook);
}

mc_status mc_merge_pair_q4(const mc_config* cfg, const mc_batch* batch, const mc_layer_q4* lm1, const mc_layer_q4* l,
                           const mc_pair_cache* out, int32_t do_retention, void* workspace, size_t workspace_bytes,
                           void* stream) {
  ApiRange range_("mc_merge_pair_q4");
  mc_status st = check_config(cfg);
  if (st != MC_OK) return st;
  if (cfg->page_size != 32) return MC_ERR_SHAPE;
  st = check_batch(cfg, batch);
  if (st != MC_OK) return st;
  if (!lm1 || !l) return MC_ERR_INVALID_ARG;
  const void* ptrs[8] = {lm1->k_codes, lm1->k_meta, lm1->v_codes, lm1->v_meta, l->k_codes, l->k_meta, l->v_codes, l->v_meta};
  for (const void* q : ptrs) {
    if (q == nullptr) return MC_ERR_INVALID_ARG;
    if (!aligned256(q)) return MC_ERR_ALIGN;
  }
  st = check_merge_common(cfg, batch, out, workspace, workspace_bytes);
  if (st != MC_OK) return st;
  return run_merge(cfg, batch, nullptr, nullptr, lm1, l, out, do_retention ? 1 : 0, workspace, (cudaStream_t)stream);
}

mc_status mc_append_pair(const mc_config* cfg, const mc_batch* batch, const mc_pair_cache* pair, const void* k_new_lm1,
                         const void* v_new_lm1, const void* k_new_l, const void* v_new_l, void* stream) {
  ApiRange range_("mc_append_pair");
  mc_status st = check_config(cfg);
  if (st != MC_OK) return st;
  st = check_batch(cfg, batch);
  if (st != MC_OK) return st;
  st = check_pair(cfg, pair);
  if (st != MC_OK) return st;
  if (!k_new_lm1 || !v_new_lm1 || !k_new_l || !v_new_l) return MC_ERR_INVALID_ARG;
  const uintptr_t al = (uintptr_t)k_new_lm1 | (uintptr_t)v_new_lm1 | (uintptr_t)k_new_l | (uintptr_t)v_new_l;
  if (al & 15u) return MC_ERR_ALIGN;
  if (cfg->cache_bits == 4)
    return launch_append_q4(cfg, batch, make_geom(cfg, batch), pair, k_new_lm1, v_new_lm1, k_new_l, v_new_l, (cudaStream_t)stream);
  return launch_append(cfg, batch, make_geom(cfg, batch), pair, k_new_lm1, v_new_lm1, k_new_l, v_new_l,
                       (cudaStream_t)stream);
}

mc_status mc_restore(const mc_config* cfg, const mc_batch* batch, const mc_pair_cache* pair, int32_t layer_sel,
                     const mc_layer_kv* dst, int32_t dst_fp32, void* stream) {
  ApiRange range_("mc_restore");
  mc_status st = check_config(cfg);
  if (st != MC_OK) return st;
  st = check_batch(cfg, batch);
  if (st != MC_OK) return st;
  st = check_pair(cfg, pair);
  if (st != MC_OK) return st;
  if (layer_sel != MC_LAYER_LM1 && layer_sel != MC_LAYER_L) return MC_ERR_INVALID_ARG;
  if (!dst || !dst->k_pool || !dst->v_pool) return MC_ERR_INVALID_ARG;
  if (!aligned256(dst->k_pool) || !aligned256(dst->v_pool)) return MC_ERR_ALIGN;
  if (batch->batch > kMaxBatchPages) return MC_ERR_SHAPE;
  if (cfg->cache_bits == 4)
    return launch_restore_q4(cfg, batch, make_geom(cfg, batch), pair, layer_sel, dst, dst_fp32 ? 1 : 0, (cudaStream_t)stream);
  return launch_restore(cfg, batch, make_geom(cfg, batch), pair, layer_sel, dst, dst_fp32 ? 1 : 0, (cudaStream_t)stream);
}

mc_status mc_decode_attn(const mc_config* cfg, const mc_batch* batch, const mc_pair_cache* pair, int32_t layer_sel,
                         const void* q, const void* k_new, const void* v_new, float sm_scale, void* out, float* lse,
                         void* workspace, size_t workspace_bytes, void* stream) {
  ApiRange range_("mc_decode_attn");
  mc_status st = check_config(cfg);
  if (st != MC_OK) return st;
  st = check_batch(cfg, batch);
  if (st != MC_OK) return st;
  st = check_pair(cfg, pair);
  if (st != MC_OK) return st;
  if (layer_sel < MC_LAYER_LM1 || layer_sel > MC_LAYER_BOTH) return MC_ERR_INVALID_ARG;
  const int n_sets = layer_sel == MC_LAYER_BOTH ? 2 : 1;
  if (n_sets * (cfg->n_q_heads / cfg->n_kv_heads) > 8) return MC_ERR_SHAPE;
  if (!q || !out) return MC_ERR_INVALID_ARG;
  if ((k_new == nullptr) != (v_new == nullptr)) return MC_ERR_INVALID_ARG;
  if (((uintptr_t)q | (uintptr_t)out | (uintptr_t)k_new | (uintptr_t)v_new) & 15u) return MC_ERR_ALIGN;
  if (workspace == nullptr || !aligned256(workspace)) return workspace ? MC_ERR_ALIGN : MC_ERR_INVALID_ARG;
  if (workspace_bytes < attn_workspace_bytes(cfg, batch, n_sets)) return MC_ERR_CAPACITY;
  return launch_decode_attn(cfg, batch, make_geom(cfg, batch), pair, layer_sel, q, k_new, v_new, sm_scale, out, lse,
                            workspace, (cudaStream_t)stream);
}

mc_status mc_decode_attn_append(const mc_config* cfg, const mc_batch* batch, const mc_pair_cache* pair, int32_t layer_sel,
                                const void* q, const void* k_new, const void* v_new, float sm_scale, void* out, float* lse,
                                const void* k_new_lm1, const void* v_new_lm1, const void* k_new_l, const void* v_new_l,
                                void* workspace, size_t workspace_bytes, void* stream) {
  ApiRange range_("mc_decode_attn_append");
  mc_status st = check_config(cfg);
  if (st != MC_OK) return st;
  st = check_batch(cfg, batch);
  if (st != MC_OK) return st;
  st = check_pair(cfg, pair);
  if (st != MC_OK) return st;
  // every check of both calls before the first launch
  if (layer_sel < MC_LAYER_LM1 || layer_sel > MC_LAYER_BOTH) return MC_ERR_INVALID_ARG;
  const int n_sets = layer_sel == MC_LAYER_BOTH ? 2 : 1;
  if (n_sets * (cfg->n_q_heads / cfg->n_kv_heads) > 8) return MC_ERR_SHAPE;
  if (!q || !out) return MC_ERR_INVALID_ARG;
  if ((k_new == nullptr) != (v_new == nullptr)) return MC_ERR_INVALID_ARG;
  if (((uintptr_t)q | (uintptr_t)out | (uintptr_t)k_new | (uintptr_t)v_new) & 15u) return MC_ERR_ALIGN;
  if (!k_new_lm1 || !v_new_lm1 || !k_new_l || !v_new_l) return MC_ERR_INVALID_ARG;
  if (((uintptr_t)k_new_lm1 | (uintptr_t)v_new_lm1 | (uintptr_t)k_new_l | (uintptr_t)v_new_l) & 15u) return MC_ERR_ALIGN;
  if (workspace == nullptr || !aligned256(workspace)) return workspace ? MC_ERR_ALIGN : MC_ERR_INVALID_ARG;
  if (workspace_bytes < attn_workspace_bytes(cfg, batch, n_sets)) return MC_ERR_CAPACITY;
  const Geom g = make_geom(cfg, batch);
  if (cfg->cache_bits == 4) {  // the 4-bit cache's append quantises whole pages: a launch of its own, after the attention
    st = launch_decode_attn(cfg, batch, g, pair, layer_sel, q, k_new, v_new, sm_scale, out, lse, workspace, (cudaStream_t)stream);
    if (st != MC_OK) return st;
    return launch_append_q4(cfg, batch, g, pair, k_new_lm1, v_new_lm1, k_new_l, v_new_l, (cudaStream_t)stream);
  }
  const AppendParams app = make_append_params(cfg, batch, g, pair, k_new_lm1, v_new_lm1, k_new_l, v_new_l);
  return launch_decode_attn(cfg, batch, g, pair, layer_sel, q, k_new, v_new, sm_scale, out, lse, workspace, (cudaStream_t)stream,
                            &app);
}

mc_status mc_merge_pair_host(const mc_config* cfg, const mc_batch* batch, const mc_layer_kv* host_lm1,
                             const mc_layer_kv* host_l, const mc_layer_kv* dev_lm1, const mc_layer_kv* dev_l,
                             const mc_pair_cache* out, int32_t do_retention, void* workspace, size_t workspace_bytes,
                             void* stream) {
  ApiRange range_("mc_merge_pair_host");
  mc_status st = check_config(cfg);
  if (st != MC_OK) return st;
  st = check_batch(cfg, batch);
  if (st != MC_OK) return st;
  if (!host_lm1 || !host_l || !dev_lm1 || !dev_l) return MC_ERR_INVALID_ARG;
  if (!host_lm1->k_pool || !host_lm1->v_pool || !host_l->k_pool || !host_l->v_pool) return MC_ERR_INVALID_ARG;
  if (!dev_lm1->k_pool || !dev_lm1->v_pool || !dev_l->k_pool || !dev_l->v_pool) return MC_ERR_INVALID_ARG;
  // every check of mc_merge_pair before the first copy: an argument error enqueues nothing
  st = check_merge_common(cfg, batch, out, workspace, workspace_bytes);
  if (st != MC_OK) return st;
  if (!aligned256(dev_lm1->k_pool) || !aligned256(dev_lm1->v_pool) || !aligned256(dev_l->k_pool) || !aligned256(dev_l->v_pool))
    return MC_ERR_ALIGN;
  const size_t pool_bytes = (size_t)batch->n_pages * cfg->n_kv_heads * cfg->page_size * kRowBytes;
  cudaStream_t s = (cudaStream_t)stream;
  MC_CUDA_CHECK(cudaMemcpyAsync(dev_lm1->k_pool, host_lm1->k_pool, pool_bytes, cudaMemcpyHostToDevice, s));
  MC_CUDA_CHECK(cudaMemcpyAsync(dev_lm1->v_pool, host_lm1->v_pool, pool_bytes, cudaMemcpyHostToDevice, s));
  MC_CUDA_CHECK(cudaMemcpyAsync(dev_l->k_pool, host_l->k_pool, pool_bytes, cudaMemcpyHostToDevice, s));
  MC_CUDA_CHECK(cudaMemcpyAsync(dev_l->v_pool, host_l->v_pool, pool_bytes, cudaMemcpyHostToDevice, s));
  return mc_merge_pair(cfg, batch, dev_lm1, dev_l, out, do_retention, workspace, workspace_bytes, stream);
}

// The device's address of pinned, device-addressable host memory; nullptr for anything else.
static const void* device_view(const void* host_ptr) {
  cudaPointerAttributes a;
  if (cudaPointerGetAttributes(&a, host_ptr) != cudaSuccess) {
    cudaGetLastError();  // pageable memory is reported as an error by older runtimes: not an error here
    return nullptr;
  }
  if (a.type != cudaMemoryTypeHost || a.devicePointer == nullptr) return nullptr;
  return a.devicePointer;
}

static void decode_io_layout(const mc_config* cfg, const mc_batch* bt, int n_sets, size_t off[6]) {
  const size_t qb = align_up((size_t)n_sets * bt->batch * cfg->n_q_heads * kRowBytes, 256);
  const size_t nb = align_up((size_t)n_sets * bt->batch * cfg->n_kv_heads * kRowBytes, 256);
  const size_t lb = align_up((size_t)n_sets * bt->batch * cfg->n_q_heads * sizeof(float), 256);
  off[0] = 0;            // q
  off[1] = qb;           // k_new
  off[2] = qb + nb;      // v_new
  off[3] = qb + 2 * nb;  // out
  off[4] = 2 * qb + 2 * nb;  // lse
  off[5] = 2 * qb + 2 * nb + lb;
}

mc_status mc_decode_io_bytes(const mc_config* cfg, const mc_batch* batch, int32_t n_query_sets, size_t* bytes) {
  mc_status st = check_config(cfg);
  if (st != MC_OK) return st;
  if (!batch || !bytes || batch->batch < 0 || (n_query_sets != 1 && n_query_sets != 2)) return MC_ERR_INVALID_ARG;
  size_t off[6];
  decode_io_layout(cfg, batch, n_query_sets, off);
  *bytes = off[5];
  return MC_OK;
}

mc_status mc_decode_attn_host(const mc_config* cfg, const mc_batch* batch, const mc_pair_cache* pair,
                              int32_t layer_sel, const void* q_host, const void* k_new_host, const void* v_new_host,
                              float sm_scale, void* out_host, float* lse_host, void* dev_io, size_t dev_io_bytes,
                              void* workspace, size_t workspace_bytes, void* stream) {
  ApiRange range_("mc_decode_attn_host");
  mc_status st = check_config(cfg);
  if (st != MC_OK) return st;
  st = check_batch(cfg, batch);
  if (st != MC_OK) return st;
  if (layer_sel < MC_LAYER_LM1 || layer_sel > MC_LAYER_BOTH) return MC_ERR_INVALID_ARG;
  if (!q_host || !out_host || !dev_io) return MC_ERR_INVALID_ARG;
  if ((k_new_host == nullptr) != (v_new_host == nullptr)) return MC_ERR_INVALID_ARG;
  if (!aligned256(dev_io)) return MC_ERR_ALIGN;
  const int n_sets = layer_sel == MC_LAYER_BOTH ? 2 : 1;
  size_t off[6];
  decode_io_layout(cfg, batch, n_sets, off);
  if (dev_io_bytes < off[5]) return MC_ERR_CAPACITY;
  char* io = (char*)dev_io;
  cudaStream_t s = (cudaStream_t)stream;
  const size_t qb = (size_t)n_sets * batch->batch * cfg->n_q_heads * kRowBytes;
  const size_t nb = (size_t)n_sets * batch->batch * cfg->n_kv_heads * kRowBytes;
  // Pinned host memory that the device can address (what cudaHostAlloc / cudaHostRegister give on a
  // unified address space) is read and written by the kernels themselves: the queries by the
  // attention kernel (prefetched a piece ahead), the new rows by one small copy kernel into the
  // staging buffer, the result by the combine kernel.  No copy engine is involved, so these small
  // transfers do not queue behind large uploads that may be running on another stream.  Any other
  // host memory goes through asynchronous copies.
  const void* q_dev = device_view(q_host);
  const void* kn_dev = k_new_host ? device_view(k_new_host) : nullptr;
  const void* vn_dev = v_new_host ? device_view(v_new_host) : nullptr;
  void* out_dev = const_cast<void*>(device_view(out_host));
  float* lse_dev = lse_host ? (float*)const_cast<void*>(device_view(lse_host)) : nullptr;
  const bool direct = q_dev && out_dev && aligned256(q_dev) && aligned256(out_dev) && (!k_new_host || (kn_dev && vn_dev)) &&
                      (!lse_host || lse_dev) && (nb % 16 == 0);
  if (direct) {
    if (k_new_host) {
      st = launch_fetch_rows(kn_dev, vn_dev, io + off[1], io + off[2], nb, s);
      if (st != MC_OK) return st;
    }
    return mc_decode_attn(cfg, batch, pair, layer_sel, q_dev, k_new_host ? io + off[1] : nullptr,
                          k_new_host ? io + off[2] : nullptr, sm_scale, out_dev, lse_dev, workspace, workspace_bytes, stream);
  }
  MC_CUDA_CHECK(cudaMemcpyAsync(io + off[0], q_host, qb, cudaMemcpyHostToDevice, s));
  if (k_new_host) {
    MC_CUDA_CHECK(cudaMemcpyAsync(io + off[1], k_new_host, nb, cudaMemcpyHostToDevice, s));
    MC_CUDA_CHECK(cudaMemcpyAsync(io + off[2], v_new_host, nb, cudaMemcpyHostToDevice, s));
  }
  st = mc_decode_attn(cfg, batch, pair, layer_sel, io + off[0], k_new_host ? io + off[1] : nullptr,
                      k_new_host ? io + off[2] : nullptr, sm_scale, io + off[3],
                      lse_host ? (float*)(io + off[4]) : nullptr, workspace, workspace_bytes, stream);
  if (st != MC_OK) return st;
  MC_CUDA_CHECK(cudaMemcpyAsync(out_host, io + off[3], qb, cudaMemcpyDeviceToHost, s));
  if (lse_host)
    MC_CUDA_CHECK(cudaMemcpyAsync(lse_host, io + off[4], (size_t)n_sets * batch->batch * cfg->n_q_heads * sizeof(float),
                                  cudaMemcpyDeviceToHost, s));
  return MC_OK;
}

mc_status mc_decode_stage_host(const mc_config* cfg, const mc_batch* batch, int32_t n_query_sets, const void* q_host,
                               const void* k_new_host, const void* v_new_host, void* dev_io, size_t dev_io_bytes, void** q_dev,
                               void** k_new_dev, void** v_new_dev, void* stream) {
  ApiRange range_("mc_decode_stage_host");
  mc_status st = check_config(cfg);
  if (st != MC_OK) return st;
  if (!batch || batch->batch < 0 || (n_query_sets != 1 && n_query_sets != 2)) return MC_ERR_INVALID_ARG;
  if (!q_host || !dev_io || !q_dev || !k_new_dev || !v_new_dev) return MC_ERR_INVALID_ARG;
  if ((k_new_host == nullptr) != (v_new_host == nullptr)) return MC_ERR_INVALID_ARG;
  if (!aligned256(dev_io)) return MC_ERR_ALIGN;
  size_t off[6];
  decode_io_layout(cfg, batch, n_query_sets, off);
  if (dev_io_bytes < off[5]) return MC_ERR_CAPACITY;
  char* io = (char*)dev_io;
  cudaStream_t s = (cudaStream_t)stream;
  const size_t qb = (size_t)n_query_sets * batch->batch * cfg->n_q_heads * kRowBytes;
  const size_t nb = (size_t)n_query_sets * batch->batch * cfg->n_kv_heads * kRowBytes;
  *q_dev = io + off[0];
  *k_new_dev = k_new_host ? io + off[1] : nullptr;
  *v_new_dev = v_new_host ? io + off[2] : nullptr;
  // device-addressable pinned memory is fetched by a kernel (no copy engine: the transfer does not queue behind
  // large uploads on other streams); anything else by asynchronous copies
  const void* src[3] = {device_view(q_host), k_new_host ? device_view(k_new_host) : nullptr,
                        v_new_host ? device_view(v_new_host) : nullptr};
  void* dst[3] = {io + off[0], io + off[1], io + off[2]};
  const size_t bytes[3] = {qb, nb, nb};
  const int n = k_new_host ? 3 : 1;
  bool direct = true;
  for (int a = 0; a < n; ++a) direct = direct && src[a] != nullptr && (((uintptr_t)src[a]) & 15u) == 0;
  if (direct) return launch_fetch3(src, dst, bytes, n, s);
  MC_CUDA_CHECK(cudaMemcpyAsync(dst[0], q_host, qb, cudaMemcpyHostToDevice, s));
  if (k_new_host) {
    MC_CUDA_CHECK(cudaMemcpyAsync(dst[1], k_new_host, nb, cudaMemcpyHostToDevice, s));
    MC_CUDA_CHECK(cudaMemcpyAsync(dst[2], v_new_host, nb, cudaMemcpyHostToDevice, s));
  }
  return MC_OK;
}

mc_status mc_decode_drain_host(const mc_config* cfg, const mc_batch* batch, int32_t n_query_sets, const void* out_dev,
                               const float* lse_dev, void* out_host, float* lse_host, void* stream) {
  ApiRange range_("mc_decode_drain_host");
  mc_status st = check_config(cfg);
  if (st != MC_OK) return st;
  if (!batch || batch->batch < 0 || (n_query_sets != 1 && n_query_sets != 2)) return MC_ERR_INVALID_ARG;
  if (!out_dev || !out_host || ((lse_dev == nullptr) != (lse_host == nullptr))) return MC_ERR_INVALID_ARG;
  const size_t rows = (size_t)n_query_sets * batch->batch * cfg->n_q_heads;
  if (rows == 0) return MC_OK;
  MC_CUDA_CHECK(cudaMemcpyAsync(out_host, out_dev, rows * kRowBytes, cudaMemcpyDeviceToHost, (cudaStream_t)stream));
  if (lse_host) MC_CUDA_CHECK(cudaMemcpyAsync(lse_host, lse_dev, rows * sizeof(float), cudaMemcpyDeviceToHost, (cudaStream_t)stream));
  return MC_OK;
}

mc_status mc_selftest_wait_timeout(const mc_pair_cache* pair, int32_t poll_limit, void* stream) {
  if (pair == nullptr || pair->status == nullptr || poll_limit <= 0) return MC_ERR_INVALID_ARG;
  return launch_wait_timeout_probe(pair->status, (uint32_t)poll_limit, (cudaStream_t)stream);
}

mc_status mc_read_status(const mc_pair_cache* pair, void* stream, int32_t* out_words) {
  if (pair == nullptr || pair->status == nullptr || out_words == nullptr) return MC_ERR_INVALID_ARG;
  MC_CUDA_CHECK(cudaMemcpyAsync(out_words, pair->status, MC_STATUS_WORDS * sizeof(int32_t), cudaMemcpyDeviceToHost,
                                (cudaStream_t)stream));
  MC_CUDA_CHECK(cudaStreamSynchronize((cudaStream_t)stream));
  if (out_words[MC_STATUS_FLAGS] & MC_FLAG_RETAIN_OVERFLOW) return MC_ERR_CAPACITY;
  if (out_words[MC_STATUS_FLAGS] != 0) return MC_ERR_DEVICE_STATUS;
  return MC_OK;
}

}  // extern "C"
