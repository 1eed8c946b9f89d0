// Internal launch interface between the C-ABI dispatch (mc_api.cu) and the kernel files.
#pragma once
#include "mc_common.cuh"

namespace mc {

// Multiprocessors of the current device (looked up once per device; the persistent grids are sized by it).
mc_status sm_count(int* n_sm);

size_t merge_workspace_bytes(const mc_config* cfg, const mc_batch* bt);
mc_status launch_merge(const mc_config* cfg, const mc_batch* bt, const Geom& g, const mc_layer_kv* lm1,
                       const mc_layer_kv* l, const mc_layer_q4* q_lm1, const mc_layer_q4* q_l, const mc_pair_cache* out,
                       int do_retention, void* workspace, cudaStream_t stream);
// Up to kMergePairsPerLaunch pairs that share the batch geometry in one launch sequence (one persistent
// merge grid over all pairs' rows, one retention pass each over all pairs' segments); the workspace
// holds merge_workspace_bytes per pair, one after the other.
// g.seq_begin / g.seq_count select the sequences the call works on.  region_rows > 0 (admission of new
// sequences): sequence b's retained entries go to the entries [b * region_rows, (b + 1) * region_rows) of the
// pool instead of one compact list for the batch, and the status words are not cleared.
constexpr int kMergePairsPerLaunch = 8;
mc_status launch_merge_pairs(const mc_config* cfg, const mc_batch* bt, const Geom& g, int n_pairs, const mc_layer_kv* const* lm1,
                             const mc_layer_kv* const* l, const mc_layer_q4* const* q_lm1, const mc_layer_q4* const* q_l,
                             const mc_pair_cache* const* out, int do_retention, void* workspace, cudaStream_t stream,
                             int region_rows = 0, const struct PrefillHook* hook = nullptr);
// With a hook (one pair), the rows of layer l come out of its projection inside launch_prefill_merge instead of
// from pools; `l` then names the pools that receive the raw rows of tokens with d > d_hint.
struct PrefillHook {
  const mc_projection* proj;
  float d_hint;
};
mc_status launch_prefill_merge(const mc_config* cfg, const mc_batch* bt, const Geom& g, const mc_projection* proj,
                               const mc_layer_kv* lm1, const mc_layer_kv* l, const mc_pair_cache* out, float d_hint,
                               cudaStream_t stream);
mc_status launch_append(const mc_config* cfg, const mc_batch* bt, const Geom& g, const mc_pair_cache* pair,
                        const void* k_new_lm1, const void* v_new_lm1, const void* k_new_l, const void* v_new_l,
                        cudaStream_t stream);
mc_status launch_restore(const mc_config* cfg, const mc_batch* bt, const Geom& g, const mc_pair_cache* pair,
                         int layer, const mc_layer_kv* dst, int dst_fp32, cudaStream_t stream);

// The 4-bit shared cache (cfg->cache_bits = 4).  The merge writes 16-bit tiles into a staging area
// (q4_stage_bytes per tensor, part of the merge workspace), which launch_q4_quantise turns into 4-bit
// tiles and residual tiles.
size_t q4_stage_bytes(const mc_config* cfg, const mc_batch* bt);
mc_status launch_q4_quantise(const mc_config* cfg, const mc_batch* bt, const Geom& g, const void* stage_k, const void* stage_v,
                             const mc_pair_cache* out, cudaStream_t stream);
mc_status launch_append_q4(const mc_config* cfg, const mc_batch* bt, const Geom& g, const mc_pair_cache* pair,
                           const void* k_new_lm1, const void* v_new_lm1, const void* k_new_l, const void* v_new_l,
                           cudaStream_t stream);
mc_status launch_restore_q4(const mc_config* cfg, const mc_batch* bt, const Geom& g, const mc_pair_cache* pair, int layer,
                            const mc_layer_kv* dst, int dst_fp32, cudaStream_t stream);

size_t attn_workspace_bytes(const mc_config* cfg, const mc_batch* bt, int n_sets);
// `append` (may be null): the decode step's append for this pair, folded into the combine launch (16-bit cache).
struct AppendParams;
mc_status launch_decode_attn(const mc_config* cfg, const mc_batch* bt, const Geom& g, const mc_pair_cache* pair,
                             int layer_sel, const void* q, const void* k_new, const void* v_new, float sm_scale,
                             void* out, float* lse, void* workspace, cudaStream_t stream, const AppendParams* append = nullptr);

// Up to three arrays (sizes multiples of 16 bytes) from device-addressable host memory into device memory, by a kernel.
mc_status launch_fetch3(const void* const* src, void* const* dst, const size_t* bytes, int n, cudaStream_t stream);
// Copies the new token's K and V rows (n bytes each, a multiple of 16) from device-addressable host
// memory into device staging with one small kernel.
mc_status launch_fetch_rows(const void* k_src, const void* v_src, void* k_dst, void* v_dst, size_t n, cudaStream_t stream);

// One warp runs into the bounded wait's limit (`limit` polls) and records it in `status`.
mc_status launch_wait_timeout_probe(int32_t* status, uint32_t limit, cudaStream_t stream);

}  // namespace mc
