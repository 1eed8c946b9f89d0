// Decode-time append (Algorithm 2 "MiniCache Decoding": merge of the step's new token pair), as a device
// function: run by append_kernel, and by the extra blocks of the attention's combine kernel when the append
// is folded into the attention call of the pair's second layer.
#pragma once
#include "mc_common.cuh"
#include "mc_retain.cuh"

namespace mc {

struct AppendParams {
  Geom g;
  const char* a_new[2];  // [batch][H][128]: K, V of layer l-1
  const char* c_new[2];
  char* e_pool[2];
  float* dist;
  float ta, tc;
  int merge_fn;
  int t_mode;
  int total_rows;  // 2 * batch * H
  int32_t* status;
  AppendKeep keep;
};

inline AppendParams make_append_params(const mc_config* cfg, const mc_batch* bt, const Geom& g, const mc_pair_cache* pair,
                                       const void* k_new_lm1, const void* v_new_lm1, const void* k_new_l, const void* v_new_l) {
  AppendParams ap;
  ap.g = g;
  ap.a_new[0] = (const char*)k_new_lm1;
  ap.a_new[1] = (const char*)v_new_lm1;
  ap.c_new[0] = (const char*)k_new_l;
  ap.c_new[1] = (const char*)v_new_l;
  ap.e_pool[0] = (char*)pair->e_k;
  ap.e_pool[1] = (char*)pair->e_v;
  ap.dist = pair->dist;
  ap.merge_fn = cfg->merge_fn;
  ap.t_mode = cfg->t_mode;
  ap.ta = (float)(1.0 - cfg->t);
  ap.tc = (float)cfg->t;
  ap.total_rows = 2 * bt->batch * cfg->n_kv_heads;
  ap.status = pair->status;
  ap.keep = make_append_keep(cfg, pair);
  return ap;
}

#if defined(__CUDACC__)
// One row (tensor, sequence, kv head) = r per half-warp; l16 = the lane's 16-byte chunk of the row.  Every lane
// of the half-warp must call it (rows past total_rows do nothing).  `wait` is called once the batch
// description has been read and before the pair cache is touched.
template <int DT, typename Wait>
__device__ __forceinline__ void append_row(const AppendParams& p, int r, int l16, Wait wait) {
  const bool ok = r < p.total_rows;
  const int rr = ok ? r : 0;
  const int H = p.g.n_kv_heads;
  const int h = rr % H;
  const int b = (rr / H) % p.g.batch;
  const int tensor = rr / (H * p.g.batch);
  // the batch description belongs to the caller (no kernel of this library writes it): where the row
  // goes is looked up before the wait on the kernel ahead in the stream
  // (a length or page id that does not fit the declared bounds is flagged after the wait -- the
  // status words belong to the pair cache -- and the row is not written)
  const int tok = p.g.seq_lens[b];
  int page = -1;
  if (tok >= 0 && tok <= p.g.max_seq_len && (tok >> p.g.page_shift) < p.g.max_pages_per_seq)
    page = p.g.block_table[(size_t)b * p.g.max_pages_per_seq + (tok >> p.g.page_shift)];
  wait();
  if (ok && !page_ok(p.g, page)) {
    if (l16 == 0) atomicOr(p.status, MC_FLAG_BAD_METADATA);
  }
  uint4 va = make_uint4(0, 0, 0, 0), vc = va;
  if (ok) {
    const size_t off = ((size_t)b * H + h) * kRowBytes + l16 * 16;
    va = *reinterpret_cast<const uint4*>(p.a_new[tensor] + off);
    vc = *reinterpret_cast<const uint4*>(p.c_new[tensor] + off);
  }
  uint4 e;
  float ga, gc, d;
  merge_row<DT>(va, vc, p.ta, p.tc, p.merge_fn, p.t_mode, e, ga, gc, d);
  const unsigned half_mask = 0xffffu << (threadIdx.x & 16);
  bool kept = false;
  if (p.keep.slack > 0) {  // (uniform over the launch)
    const int seg = (tensor * p.g.batch + b) * H + h;
    bool keep = ok && page_ok(p.g, page) && append_keeps(p.keep, seg, d);
    if (p.keep.union_kv) {
      // one set for keys and values: the other tensor's rule, on its own new rows, counts as well
      uint4 oa = make_uint4(0, 0, 0, 0), oc = oa;
      if (ok) {
        const size_t off = ((size_t)b * H + h) * kRowBytes + l16 * 16;
        oa = *reinterpret_cast<const uint4*>(p.a_new[1 - tensor] + off);
        oc = *reinterpret_cast<const uint4*>(p.c_new[1 - tensor] + off);
      }
      uint4 e_o;
      float ga_o, gc_o, d_o;
      merge_row<DT>(oa, oc, p.ta, p.tc, p.merge_fn, p.t_mode, e_o, ga_o, gc_o, d_o);
      keep = keep || (ok && page_ok(p.g, page) && append_keeps(p.keep, ((1 - tensor) * p.g.batch + b) * H + h, d_o));
    }
    keep = __shfl_sync(half_mask, (int)keep, threadIdx.x & 16) != 0;  // (one decision per half-warp)
    if (keep) kept = append_retain(p.keep, seg, tok, l16, va, vc, p.status);
  }
  if (!ok || !page_ok(p.g, page)) return;
  if (kept) ga = gc = -0.f;  // served from its raw rows (the mark retain_compact_kernel leaves as well)
  const int tk = tok & (p.g.page_size - 1);
  const size_t ph = (size_t)page * H + h;
  char* tile = p.e_pool[tensor] + ph * tile_bytes(p.g.page_size);
  *reinterpret_cast<uint4*>(tile + tk * kRowBytes + chunk_pos(tk, l16) * 16) = e;
  if (l16 == 0) {
    float* sc = reinterpret_cast<float*>(tile + p.g.page_size * kRowBytes) + tk;
    sc[0] = ga;
    sc[p.g.page_size] = gc;
    p.dist[(ph * 2 + tensor) * p.g.page_size + tk] = d;
  }
}
#endif

}  // namespace mc
