// Eq. 4's decision for one token, and the decode-time extension of it: a token appended by
// Algorithm 2 "MiniCache Decoding" is held against the threshold of its segment's prefill tokens
// (d_min, d_max as stored when the pair was merged) and, if the rule keeps it, joins the segment's
// retained list in one of the free entries laid out behind it.
#pragma once
#include "mc_common.cuh"

namespace mc {

// Retention decision of one token; the threshold is formed in double from the fp32 extremes.
__device__ __forceinline__ bool keep_token(float d, float dmin, float dmax, double gamma, int mode) {
  const double lo = dmin, hi = dmax;
  if (mode == MC_RETAIN_DISTINCT) return (double)d > hi - (hi - lo) * gamma;
  return (double)d < lo + (hi - lo) * gamma;
}

struct AppendKeep {
  const float* seg_minmax;
  int32_t* ret_count;
  const int32_t* ret_offset;
  int32_t* ret_index;
  char* ret_rows;
  int64_t ret_capacity;
  int32_t* ret_prefix;
  int ret_prefix_stride;
  double gamma;
  int mode;
  int union_kv;
  int slack;  // 0: appended tokens are never kept
};

inline AppendKeep make_append_keep(const mc_config* cfg, const mc_pair_cache* pair) {
  AppendKeep k;
  k.seg_minmax = pair->seg_minmax;
  k.ret_count = pair->ret_count;
  k.ret_offset = pair->ret_offset;
  k.ret_index = pair->ret_index;
  k.ret_rows = (char*)pair->ret_rows;
  k.ret_capacity = pair->ret_capacity;
  k.ret_prefix = pair->ret_prefix;
  k.ret_prefix_stride = (int)pair->ret_prefix_stride;
  k.gamma = cfg->gamma;
  k.mode = cfg->retain_mode;
  k.union_kv = cfg->retain_union;
  // (without a pool there is nowhere to keep a token)
  k.slack = pair->ret_capacity > 0 && pair->ret_index && pair->ret_rows ? cfg->append_slack : 0;
  return k;
}

// Does Eq. 4, with the stored extremes of segment `seg`, keep a token of distance d?  (A segment
// without prefill tokens has the extremes (+inf, 0): every comparison with its threshold is false.)
__device__ __forceinline__ bool append_keeps(const AppendKeep& k, int seg, float d) {
  if (k.slack <= 0 || !(k.gamma > 0.0) || k.mode == MC_RETAIN_TOPK) return false;
  return keep_token(d, k.seg_minmax[2 * seg], k.seg_minmax[2 * seg + 1], k.gamma, k.mode);
}

// Half-warp (lane l16 holds chunk l16 of both raw rows): appends token `tok` to the retained list of
// `seg`.  Returns false, with the overflow flag set, when the segment has no free entry left (the
// entry behind the list then belongs to the next segment, or lies past the pool); the caller merges
// the token instead.  All sixteen lanes return the same value.
__device__ __forceinline__ bool append_retain(const AppendKeep& k, int seg, int tok, int l16, uint4 va, uint4 vc,
                                              int32_t* status) {
  const int cnt = k.ret_count[seg];
  const int off = k.ret_offset[seg];
  const int64_t pos = (int64_t)off + cnt;
  const bool room = off >= 0 && pos < k.ret_capacity && k.ret_index[pos] == -1;
  if (!room) {
    if (l16 == 0) atomicOr(&status[MC_STATUS_FLAGS], MC_FLAG_RETAIN_OVERFLOW);
    return false;
  }
  char* r0 = k.ret_rows + (size_t)pos * kRetEntryBytes;
  char* r1 = k.ret_rows + ((size_t)k.ret_capacity + pos) * kRetEntryBytes;
  *reinterpret_cast<uint4*>(r0 + l16 * 16) = va;
  *reinterpret_cast<uint4*>(r1 + l16 * 16) = vc;
  // entry j of the prefix table counts the retained tokens before token 128 j
  int32_t* prefix = k.ret_prefix + (size_t)seg * k.ret_prefix_stride;
  for (int j = (tok >> 7) + 1 + l16; j < k.ret_prefix_stride; j += 16) prefix[j] += 1;
  __syncwarp(0xffffu << (threadIdx.x & 16));  // every lane has read ret_index[pos] and ret_count
  if (l16 == 0) {
    *reinterpret_cast<int4*>(r0 + kRowBytes) = make_int4(tok, 0, 0, 0);
    *reinterpret_cast<int4*>(r1 + kRowBytes) = make_int4(tok, 0, 0, 0);
    k.ret_index[pos] = tok;
    k.ret_count[seg] = cnt + 1;
    atomicAdd(&status[MC_STATUS_RETAINED_TOTAL], 1);
  }
  return true;
}

}  // namespace mc
