// Cross-layer merge of one layer pair (Algorithm 2 "MiniCache Prefill"):
//   merge_kernel      Eq. 2 magnitudes, angle, Eq. 3 SLERP direction, distance d = Omega / pi,
//                     per-segment d_min / d_max
//   retain_*          Eq. 4 retention set: count, scan, ordered compaction + raw-row gather
//   append_kernel     the decode-time merge of one new token per sequence
#include <algorithm>

#include "mc_common.cuh"
#include "mc_kernels.h"
#include "mc_items.cuh"
#include "mc_pipe.cuh"
#include "mc_retain.cuh"
#include "mc_append.cuh"

namespace mc {

constexpr int kRowsPerItem = 64;  // rows of one page per work item
constexpr int kMergeStages = 3;
constexpr int kMergeStageBytes = 2 * kRowsPerItem * kRowBytes;  // the item's rows of layer l-1, then of layer l
constexpr int kMergeWarps = 8;
constexpr int kMergeThreads = kMergeWarps * 32;
constexpr int kMergeCtasPerSm = 2;
constexpr int kMergeMaxBatchSmem = kMaxBatchPages;
constexpr int kQ4RowBytes = 64;                              // 128 four-bit codes
constexpr int kQ4CodesBytes = kRowsPerItem * kQ4RowBytes;    // one layer's codes of an item
constexpr int kQ4MetaBytes = kRowsPerItem * 16;              // one layer's (scale, zero) pairs of an item

constexpr int kMaxMergePairs = 8;  // layer pairs one launch sequence can merge (they share the batch geometry)

struct MergePair {
  const char* a_pool[2];  // layer l-1: K, V
  const char* c_pool[2];  // layer l:   K, V
  const char* a_meta[2];  // 4-bit layers: (scale, zero) pairs; a_pool / c_pool then hold the codes
  const char* c_meta[2];
  char* e_pool[2];  // compressed tiles (see tile_bytes)
  float* dist;
  unsigned* seg_minmax;  // [seg][2] float bits (d >= 0, so unsigned order = float order)
  int32_t* status;
};

struct MergeParams {
  Geom g;
  MergePair pr[kMaxMergePairs];
  int n_pairs;
  float ta, tc;
  int merge_fn;
  int t_mode;
  int items_per_page;
};

// Sum of squares of the two 16-bit values of a packed word, accumulated in fp32 by the
// mixed-precision FMA of sm_100 (no conversion instructions).
template <int DT>
__device__ __forceinline__ float sq_acc(uint32_t w, float acc) {
  unsigned short lo, hi;
  asm("mov.b32 {%0, %1}, %2;" : "=h"(lo), "=h"(hi) : "r"(w));
  if (DT == MC_F16) {
    asm("fma.rn.f32.f16 %0, %1, %1, %0;" : "+f"(acc) : "h"(lo));
    asm("fma.rn.f32.f16 %0, %1, %1, %0;" : "+f"(acc) : "h"(hi));
  } else {
    asm("fma.rn.f32.bf16 %0, %1, %1, %0;" : "+f"(acc) : "h"(lo));
    asm("fma.rn.f32.bf16 %0, %1, %1, %0;" : "+f"(acc) : "h"(hi));
  }
  return acc;
}

// Sum over the 4 lanes that share one row.
__device__ __forceinline__ float sum4(float v) {
  v += __shfl_xor_sync(0xffffffffu, v, 1);
  v += __shfl_xor_sync(0xffffffffu, v, 2);
  return v;
}

// One merged row held by a quad of lanes: lane k owns the 16-byte chunks k, k + 4, k + 8, k + 12 of
// a (layer l-1) and c (layer l), 32 channels each.  Arithmetic in fp32, two channels per
// instruction (packed f32x2).  Every lane of the quad returns the row's scalars.
template <int DT>
__device__ __forceinline__ void merge_row_core(const float2 (&a)[16], const float2 (&c)[16], float ta, float tc, int fn, int t_mode,
                                               uint4 (&e_out)[4], float& g_a, float& g_c, float& d_out) {
  float2 aa2 = make_float2(0.f, 0.f), cc2 = aa2, aa3 = aa2, cc3 = aa2;
#pragma unroll
  for (int i = 0; i < 16; i += 2) {
    aa2 = __ffma2_rn(a[i], a[i], aa2);
    cc2 = __ffma2_rn(c[i], c[i], cc2);
    aa3 = __ffma2_rn(a[i + 1], a[i + 1], aa3);
    cc3 = __ffma2_rn(c[i + 1], c[i + 1], cc3);
  }
  const float aa = sum4((aa2.x + aa2.y) + (aa3.x + aa3.y)), cc = sum4((cc2.x + cc2.y) + (cc3.x + cc3.y));
  const float ia = aa > 0.f ? rsqrtf(aa) : 0.f;
  const float ic = cc > 0.f ? rsqrtf(cc) : 0.f;
  // |u - v|^2 = |a - (|a| / |c|) c|^2 / |a|^2, formed channel by channel (no cancellation at small
  // angles); |u + v|^2 = 4 - |u - v|^2 is as good until the two directions come close to opposite,
  // where it is formed the same way
  const float ia_sq = ia * ia;
  const float nr = -(aa * ia) * ic;  // -|a| / |c|
  const float2 ia2 = make_float2(ia, ia), nr2 = make_float2(nr, nr);
  float2 sm2 = make_float2(0.f, 0.f), sm3 = sm2;
#pragma unroll
  for (int i = 0; i < 16; i += 2) {
    const float2 dm = __ffma2_rn(c[i], nr2, a[i]);
    const float2 dn = __ffma2_rn(c[i + 1], nr2, a[i + 1]);
    sm2 = __ffma2_rn(dm, dm, sm2);
    sm3 = __ffma2_rn(dn, dn, sm3);
  }
  const float sm = sum4((sm2.x + sm2.y) + (sm3.x + sm3.y)) * ia_sq;
  float sp = 4.0f - sm;
  if (__any_sync(0xffffffffu, sm > 3.5f)) {
    const float2 ic2 = make_float2(ic, ic);
    float2 sp2 = make_float2(0.f, 0.f);
#pragma unroll
    for (int i = 0; i < 16; ++i) {
      const float2 dp = __ffma2_rn(c[i], ic2, __fmul2_rn(a[i], ia2));
      sp2 = __ffma2_rn(dp, dp, sp2);
    }
    const float spx = sum4(sp2.x + sp2.y);
    if (sm > 3.5f) sp = spx;
  }
  row_t(t_mode, aa, cc, ta, tc);
  RowScalars s = slerp_scalars(aa, cc, sm, fmaxf(sp, 0.f), ta, tc);
  if (fn != MC_MERGE_SLERP) {  // one vector for both layers: direction of the mean, one magnitude
    float2 m2 = make_float2(0.f, 0.f);
#pragma unroll
    for (int i = 0; i < 16; ++i) {
      const float2 h = make_float2(a[i].x + c[i].x, a[i].y + c[i].y);
      m2 = __ffma2_rn(h, h, m2);
    }
    const float mm = 0.25f * sum4(m2.x + m2.y);
    const float im = mm > 0.f ? rsqrtf(mm) : 0.f;
    s.fa = s.fc = 0.5f * im;
    s.na = s.nc = fn == MC_MERGE_FMAX ? fmaxf(s.na, s.nc) : mm * im;
  }
  const float2 fa2 = make_float2(s.fa, s.fa), fc2 = make_float2(s.fc, s.fc);
  float ee4[4] = {0.f, 0.f, 0.f, 0.f};
  uint32_t w[16];
#pragma unroll
  for (int i = 0; i < 16; ++i) {
    const float2 x = __ffma2_rn(a[i], fa2, __fmul2_rn(c[i], fc2));
    w[i] = Elem<DT>::pack(x.x, x.y);
    ee4[i & 3] = sq_acc<DT>(w[i], ee4[i & 3]);  // the stored value: Eq. 2 divides by its length
  }
  const float ee = sum4((ee4[0] + ee4[1]) + (ee4[2] + ee4[3]));
  const float il = ee > 0.f ? rsqrtf(ee) : 0.f;
#pragma unroll
  for (int i = 0; i < 4; ++i) e_out[i] = make_uint4(w[4 * i], w[4 * i + 1], w[4 * i + 2], w[4 * i + 3]);
  g_a = s.na * il;
  g_c = s.nc * il;
  d_out = s.d;
}

// Work item of the merge: 64 consecutive rows of one page (rows of a page are [head][token], so an
// item is a contiguous 16 KB block in each layer's pool).  Flattened order: tensor, sequence, page
// slot, row group -- row group fastest.
// Persistent merge kernel.  The items' rows of both layers are streamed into a ring of shared-memory
// stages with bulk asynchronous copies (two 16 KB copies per stage), issued two items ahead by lane 0
// of warp 0; the eight warps take a row per quad of lanes out of shared memory, release the stage,
// and do Eq. 2 / Eq. 3 in registers.  The bytes in flight are set by the ring, not by registers or
// occupancy.  (Eight warps, not nine with a dedicated producer: two CTAs of nine warps do not fit
// the register file of an SM sub-partition.)
template <int DT>
__device__ __forceinline__ void merge_row_quad(const uint4 (&ra)[4], const uint4 (&rc)[4], float ta, float tc, int fn, int t_mode,
                                               uint4 (&e_out)[4], float& g_a, float& g_c, float& d_out) {
  float2 a[16], c[16];
#pragma unroll
  for (int i = 0; i < 4; ++i) {
    a[4 * i] = Elem<DT>::unpack(ra[i].x);
    a[4 * i + 1] = Elem<DT>::unpack(ra[i].y);
    a[4 * i + 2] = Elem<DT>::unpack(ra[i].z);
    a[4 * i + 3] = Elem<DT>::unpack(ra[i].w);
    c[4 * i] = Elem<DT>::unpack(rc[i].x);
    c[4 * i + 1] = Elem<DT>::unpack(rc[i].y);
    c[4 * i + 2] = Elem<DT>::unpack(rc[i].z);
    c[4 * i + 3] = Elem<DT>::unpack(rc[i].w);
  }
  merge_row_core<DT>(a, c, ta, tc, fn, t_mode, e_out, g_a, g_c, d_out);
}

// 32 consecutive 4-bit codes (16 bytes; channel 2i in the low nibble of byte i) to values
// code * scale + zero, four channels at a time.  `meta` points at the lane's (scale, zero) binary16 pairs in
// shared memory: one pair per channel (keys, per_channel) or a single pair for all 32 (values, one group
// per token).  Position j of the output holds the channels [4 c, 4 c + 4) of the lane's 32 with
// c = (j + rot) & 7: for the keys the four lanes of a quad read their 32 parameter words from addresses a
// multiple of 32 words apart, so each lane starts at a different chunk (rot = 2 * lane-in-quad) and the
// 16-byte loads of a quad fall into different banks; the arithmetic that follows does not care about the
// order, only the store addresses do.
// A group of four nibbles becomes two pairs of exact binary16 integers on the way (nibble OR-ed into
// the mantissa of 1024, 1024 subtracted), and value = code * scale + zero is ONE mixed-precision FMA
// (binary16 x binary16 + binary32 -> binary32: exact product, one rounding).
__device__ __forceinline__ float h2f(unsigned short h) {
  float r;
  asm("{\n\t.reg .b16 one;\n\tmov.b16 one, 0x3C00;\n\tfma.rn.f32.f16 %0, %1, one, 0f00000000;\n\t}" : "=f"(r) : "h"(h));
  return r;
}
__device__ __forceinline__ float fma_hhf(unsigned short a, unsigned short b, float c) {
  float r;
  asm("fma.rn.f32.f16 %0, %1, %2, %3;" : "=f"(r) : "h"(a), "h"(b), "f"(c));
  return r;
}
__device__ __forceinline__ void dequant32(const uint4& codes, const uint32_t* meta, bool per_channel, int rot, float2 (&out)[16]) {
  const __half2 k1024 = __half2half2(__ushort_as_half((unsigned short)0x6400));
  unsigned short s_one = 0;
  float z_one = 0.f;
  if (!per_channel) {
    const uint32_t m = meta[0];
    s_one = (unsigned short)(m & 0xffffu);
    z_one = h2f((unsigned short)(m >> 16));
  }
#pragma unroll
  for (int j = 0; j < 8; ++j) {
    const int c = (j + rot) & 7;
    // the 16 bits of codes of chunk c: half (c & 1) of word (c >> 1)
    const uint32_t wd = (c & 4) ? ((c & 2) ? codes.w : codes.z) : ((c & 2) ? codes.y : codes.x);
    const uint32_t h16 = (wd >> ((c & 1) << 4)) & 0xffffu;
    // nibbles 0, 1 at bits 0 and 16; nibbles 2, 3 at bits 8 and 24: the low half as it is, the high half from a copy
    // shifted up by 12 bits
    const uint32_t t = __byte_perm(h16, h16 << 12, 0x7610);
    uint32_t p01 = (t & 0x000F000Fu) | 0x64006400u, p23 = ((t >> 8) & 0x000F000Fu) | 0x64006400u;
    const __half2 c01 = __hsub2(*reinterpret_cast<__half2*>(&p01), k1024), c23 = __hsub2(*reinterpret_cast<__half2*>(&p23), k1024);
    const unsigned short n0 = __half_as_ushort(__low2half(c01)), n1 = __half_as_ushort(__high2half(c01));
    const unsigned short n2 = __half_as_ushort(__low2half(c23)), n3 = __half_as_ushort(__high2half(c23));
    if (per_channel) {
      const uint4 m = *reinterpret_cast<const uint4*>(meta + 4 * c);  // (scale, zero) of the chunk's four channels
      out[2 * j] = make_float2(fma_hhf(n0, (unsigned short)(m.x & 0xffffu), h2f((unsigned short)(m.x >> 16))),
                               fma_hhf(n1, (unsigned short)(m.y & 0xffffu), h2f((unsigned short)(m.y >> 16))));
      out[2 * j + 1] = make_float2(fma_hhf(n2, (unsigned short)(m.z & 0xffffu), h2f((unsigned short)(m.z >> 16))),
                                   fma_hhf(n3, (unsigned short)(m.w & 0xffffu), h2f((unsigned short)(m.w >> 16))));
    } else {
      out[2 * j] = make_float2(fma_hhf(n0, s_one, z_one), fma_hhf(n1, s_one, z_one));
      out[2 * j + 1] = make_float2(fma_hhf(n2, s_one, z_one), fma_hhf(n3, s_one, z_one));
    }
  }
}

template <int DT, bool Q4IN>
__global__ void __launch_bounds__(kMergeThreads, kMergeCtasPerSm) merge_kernel(const __grid_constant__ MergeParams p) {
  grid_dep_wait();
  grid_dep_launch();
  extern __shared__ unsigned char smem_raw[];
  unsigned char* smem = reinterpret_cast<unsigned char*>((reinterpret_cast<uintptr_t>(smem_raw) + 127) & ~uintptr_t(127));
  unsigned char* stages = smem;
  int* page_s = reinterpret_cast<int*>(smem + kMergeStages * kMergeStageBytes);  // [kMergeStages] page id of the staged item
  int* len_s = page_s + kMergeStages;                                            // [batch]
  int* pre_s = len_s + kMergeMaxBatchSmem;                                       // [batch + 1] pages before each sequence
  volatile int* s_abort = pre_s + kMergeMaxBatchSmem + 1;
  uint64_t* bars = reinterpret_cast<uint64_t*>((reinterpret_cast<uintptr_t>(s_abort + 1) + 7) & ~uintptr_t(7));
  const uint32_t full0 = smem_u32(bars), empty0 = full0 + 8 * kMergeStages;
  const uint32_t stage0 = smem_u32(stages);
  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  const int ps = p.g.page_size, H = p.g.n_kv_heads;
  const int rows_in_page = H * ps;

  if (tid == 0) {
    for (int s = 0; s < kMergeStages; ++s) {
      mbar_init(full0 + 8 * s, 1);
      mbar_init(empty0 + 8 * s, kMergeWarps);
    }
    *s_abort = 0;
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  // (what concerns the batch as a whole -- a length outside its bound, a wait that ran out -- is
  // recorded in the first pair's status words)
  int32_t* const status0 = p.pr[0].status;
  const int n_slots = 2 * p.n_pairs;  // item order: pair, tensor, page, row group
  page_prefix(p.g, len_s, pre_s, kMergeThreads, status0);
  const int* lens = len_s;
  const int P_all = pre_s[p.g.batch];
  const int ipp = p.items_per_page;
  const int stride = gridDim.x;
  const int s_pg = stride / ipp, s_grp = stride - s_pg * ipp;

  // a page id outside the pools comes back as -1: its item streams page 0 instead (any valid
  // memory) and writes nothing
  auto page_of = [&](const PageItem& m) { return m.tensor < n_slots ? checked_page(p.g, m.b, m.pslot, p.pr[m.tensor >> 1].status) : 0; };
  // lane 0 of warp 0: copy item j (the j-th item of this CTA) into stage j % kMergeStages
  auto issue = [&](int j, const PageItem& m, int page_id) -> bool {
    const int s = j % kMergeStages;
    if (j >= kMergeStages && !mbar_wait(empty0 + 8 * s, ((j / kMergeStages) - 1) & 1, s_abort, status0)) return false;
    const MergePair& P = p.pr[m.tensor >> 1];
    const int ts = m.tensor & 1;
    const int rows_item = min(kRowsPerItem, rows_in_page - m.grp * kRowsPerItem);
    const uint32_t bar = full0 + 8 * s;
    page_s[s] = page_id;
    const int page = max(page_id, 0);
    const size_t row0 = (size_t)page * rows_in_page + m.grp * kRowsPerItem;
    if (!Q4IN) {
      const uint32_t bytes = (uint32_t)rows_item * kRowBytes;
      mbar_expect_tx(bar, 2 * bytes);
      bulk_load(stage0 + s * kMergeStageBytes, P.a_pool[ts] + row0 * kRowBytes, bytes, bar);
      bulk_load(stage0 + s * kMergeStageBytes + kRowsPerItem * kRowBytes, P.c_pool[ts] + row0 * kRowBytes, bytes, bar);
    } else {
      // 4-bit layers: 64 bytes of codes per row; (scale, zero) pairs per channel and head (keys, a
      // group = the page's 32 tokens) or per token and 32 channels (values)
      const uint32_t cbytes = (uint32_t)rows_item * kQ4RowBytes;
      const uint32_t mbytes = ts ? (uint32_t)rows_item * 16u : (uint32_t)(rows_item / 32) * 512u;
      const size_t moff = ts ? row0 * 16 : (row0 / 32) * 512;
      mbar_expect_tx(bar, 2 * (cbytes + mbytes));
      const uint32_t sb = stage0 + s * kMergeStageBytes;
      bulk_load(sb, P.a_pool[ts] + row0 * kQ4RowBytes, cbytes, bar);
      bulk_load(sb + kQ4CodesBytes, P.c_pool[ts] + row0 * kQ4RowBytes, cbytes, bar);
      bulk_load(sb + 2 * kQ4CodesBytes, P.a_meta[ts] + moff, mbytes, bar);
      bulk_load(sb + 2 * kQ4CodesBytes + kQ4MetaBytes, P.c_meta[ts] + moff, mbytes, bar);
    }
    return true;
  };

  PageItem m;
  page_item_init(m, blockIdx.x, ipp, P_all, pre_s, n_slots);
  // warp 0 looks two items ahead (and loads page ids three ahead: a demand load takes microseconds
  // while the copies saturate the memory system)
  PageItem m1 = m, m2 = m, m3 = m;
  int pg2 = 0, pg3 = 0;
  if (warp == 0) {
    page_item_advance(m1, s_pg, s_grp, ipp, P_all, pre_s, n_slots);
    m2 = m1;
    page_item_advance(m2, s_pg, s_grp, ipp, P_all, pre_s, n_slots);
    m3 = m2;
    page_item_advance(m3, s_pg, s_grp, ipp, P_all, pre_s, n_slots);
    const int pg0 = page_of(m), pg1 = page_of(m1);
    pg2 = page_of(m2);
    pg3 = page_of(m3);
    if (lane == 0) {
      if (m.tensor < n_slots) issue(0, m, pg0);
      if (m1.tensor < n_slots) issue(1, m1, pg1);
    }
  }

  const int quad = tid >> 2, k = tid & 3;
  // Distance extremes: every lane keeps the running d_min / d_max of its own rows while the warp's items
  // keep falling into the same segment (consecutive items of a CTA usually do: all CTAs work on one
  // sequence at a time); only when the segment changes are the lanes reduced and one atomic pair sent.
  // (One atomic pair per warp and item on a segment's few addresses queues up in the memory system, and
  // a per-item warp reduction is a chain of shuffles at the end of every item.)
  int run_key = -1;             // (slot, sequence, head) of the running extremes
  unsigned* run_ptr = nullptr;  // its d_min / d_max words
  float run_min = __int_as_float(0x7f800000), run_max = 0.f;
  auto flush_extremes = [&]() {
    if (run_key < 0) return;
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) {
      run_min = fminf(run_min, __shfl_xor_sync(0xffffffffu, run_min, o));
      run_max = fmaxf(run_max, __shfl_xor_sync(0xffffffffu, run_max, o));
    }
    if (lane == 0 && run_min != __int_as_float(0x7f800000)) {  // (some row of the run was a cached token)
      atomicMin(run_ptr, __float_as_uint(run_min));
      atomicMax(run_ptr + 1, __float_as_uint(run_max));
    }
  };
  for (int it = 0; m.tensor < n_slots; ++it) {
    if (warp == 0) {
      // item it + 2 goes into the stage that item it - 1 has just left
      int good = 1;
      if (lane == 0 && m2.tensor < n_slots) good = issue(it + 2, m2, pg2) ? 1 : 0;
      good = __shfl_sync(0xffffffffu, good, 0);
      if (!good) break;
      m2 = m3;
      pg2 = pg3;
      page_item_advance(m3, s_pg, s_grp, ipp, P_all, pre_s, n_slots);
      pg3 = page_of(m3);
    }
    const int s = it % kMergeStages;
    if (!mbar_wait(full0 + 8 * s, (it / kMergeStages) & 1, s_abort, status0)) break;
    const MergePair& P = p.pr[m.tensor >> 1];
    const int ts = m.tensor & 1;
    const int page = page_s[s];
    const int n = lens[m.b];
    const int row = m.grp * kRowsPerItem + quad;  // one row per quad of lanes; a warp = 8 consecutive rows of one head
    const int head = row >> p.g.page_shift;
    const int tk = row & (ps - 1);
    const bool valid = page >= 0 && row < rows_in_page && m.pslot * ps + tk < n;
    uint4 e[4];
    float g_a, g_c, d;
    int ci[4];
    if (!Q4IN) {
      // lane k owns the 16-byte chunks k, k + 4, k + 8, k + 12; odd rows fetch them in the order that
      // keeps the two rows of a quarter-warp in different bank groups
      const unsigned char* sa = stages + s * kMergeStageBytes + quad * kRowBytes;
      const unsigned char* sc = sa + kRowsPerItem * kRowBytes;
      uint4 va[4], vc[4];
#pragma unroll
      for (int x = 0; x < 4; ++x) {
        ci[x] = ((x ^ (quad & 1)) << 2) + k;
        va[x] = *reinterpret_cast<const uint4*>(sa + ci[x] * 16);
        vc[x] = *reinterpret_cast<const uint4*>(sc + ci[x] * 16);
      }
      if (!valid) {
#pragma unroll
        for (int x = 0; x < 4; ++x) va[x] = vc[x] = make_uint4(0, 0, 0, 0);  // never computed on: page tail
      }
      __syncwarp();
      if (lane == 0) mbar_arrive(empty0 + 8 * s);  // the stage is in registers now
      merge_row_quad<DT>(va, vc, p.ta, p.tc, p.merge_fn, p.t_mode, e, g_a, g_c, d);
    } else {
      // lane k owns channels [32 k, 32 k + 32): 16 bytes of codes = the 16-byte chunks 4 k .. 4 k + 3 of the output row
      const unsigned char* sb = stages + s * kMergeStageBytes;
      const uint4 qa = *reinterpret_cast<const uint4*>(sb + quad * kQ4RowBytes + k * 16);
      const uint4 qc = *reinterpret_cast<const uint4*>(sb + kQ4CodesBytes + quad * kQ4RowBytes + k * 16);
      const bool per_channel = ts == 0;
      const int mo = per_channel ? ((quad >> 5) * 128 + 32 * k) : (quad * 4 + k);  // in (scale, zero) pairs
      const uint32_t* ma = reinterpret_cast<const uint32_t*>(sb + 2 * kQ4CodesBytes) + mo;
      const uint32_t* mc = reinterpret_cast<const uint32_t*>(sb + 2 * kQ4CodesBytes + kQ4MetaBytes) + mo;
      float2 a[16], c[16];
      const int rot = per_channel ? 2 * k : 0;
      dequant32(qa, ma, per_channel, rot, a);
      dequant32(qc, mc, per_channel, rot, c);
      if (!valid) {
#pragma unroll
        for (int x = 0; x < 16; ++x) a[x] = c[x] = make_float2(0.f, 0.f);
      }
#pragma unroll
      for (int x = 0; x < 4; ++x) ci[x] = 4 * k + ((x + (rot >> 1)) & 3);  // output chunk x holds the 8 channels of these two groups
      __syncwarp();
      if (lane == 0) mbar_arrive(empty0 + 8 * s);
      merge_row_core<DT>(a, c, p.ta, p.tc, p.merge_fn, p.t_mode, e, g_a, g_c, d);
    }
    if (valid) {
      char* tile = P.e_pool[ts] + ((size_t)page * H + head) * tile_bytes(ps);
#pragma unroll
      for (int x = 0; x < 4; ++x) st_stream16(tile + tk * kRowBytes + chunk_pos(tk, ci[x]) * 16, e[x]);
      if (k == 0) {
        float* scp = reinterpret_cast<float*>(tile + ps * kRowBytes) + tk;
        scp[0] = g_a;
        scp[ps] = g_c;
        P.dist[(((size_t)page * H + head) * 2 + ts) * ps + tk] = d;
      }
    }
    const int row_w = m.grp * kRowsPerItem + warp * 8;  // the warp's 8 rows lie in one head
    if (row_w < rows_in_page) {
      const int head_w = row_w >> p.g.page_shift;
      const int key = (m.tensor * p.g.batch + m.b) * H + head_w;
      if (key != run_key) {
        flush_extremes();
        run_key = key;
        run_ptr = P.seg_minmax + 2 * ((ts * p.g.batch + m.b) * H + head_w);
        run_min = __int_as_float(0x7f800000);
        run_max = 0.f;
      }
      if (valid) {
        run_min = fminf(run_min, d);
        run_max = fmaxf(run_max, d);
      }
    }
    page_item_advance(m, s_pg, s_grp, ipp, P_all, pre_s, n_slots);
  }
  flush_extremes();
  if (*s_abort) {
    for (int x = 0; x < 2000; ++x) __nanosleep(1000);  // let copies in flight land before the CTA's memory is released
  }
}

// ---------------------------------------------------------------------------------------------
// Retention (Eq. 4)
// ---------------------------------------------------------------------------------------------
constexpr int kChunk = 1024;  // tokens per retention work item
constexpr int kRetThreads = 256;

struct RetainParams {
  Geom g;
  const char* a_pool[2];
  const char* c_pool[2];
  const char* a_meta[2];  // 4-bit layers only
  const char* c_meta[2];
  int q4;                 // the layers are 4-bit: raw rows are de-quantised (exactly) into the storage type
  int dtype;
  char* e_pool[2];
  const float* dist;
  const float* seg_minmax;
  int32_t* chunk_count;   // workspace [nseg][chunks_per_seg]
  int32_t* chunk_offset;  // workspace [nseg][chunks_per_seg]
  int32_t* chunk_eq;      // workspace [nseg][chunks_per_seg], top-k mode: tokens equal to the k-th largest d (count, then count before the chunk)
  uint32_t* seg_sel;      // workspace [nseg][2], top-k mode: bits of the k-th largest d, how many tokens equal to it are kept
  int32_t* ret_count;
  int32_t* ret_offset;
  int32_t* ret_index;
  char* ret_rows;
  int64_t ret_capacity;
  int32_t* status;
  int32_t* ret_prefix;
  int ret_prefix_stride;
  int chunks_per_seg;
  int nseg;
  int mode;
  int do_retention;
  int union_kv;  // one set for keys and values: a token the other tensor's rule keeps is kept here too
  int region_rows;  // admission: entries of the retained pool each sequence owns (0: one compact list for the batch)
  int slack;        // free entries behind every segment's list, for tokens kept at decode time
  float d_hint;     // fused prefill: raw layer-l rows exist only for tokens with d > d_hint (< 0: for all)
  double gamma;
};

// The part of RetainParams that differs from pair to pair when several pairs are merged at once.
struct RetainPair {
  const char* a_pool[2];
  const char* c_pool[2];
  const char* a_meta[2];
  const char* c_meta[2];
  char* e_pool[2];
  const float* dist;
  const float* seg_minmax;
  int32_t* chunk_count;
  int32_t* chunk_offset;
  int32_t* chunk_eq;
  uint32_t* seg_sel;
  int32_t* ret_count;
  int32_t* ret_offset;
  int32_t* ret_index;
  char* ret_rows;
  int64_t ret_capacity;
  int32_t* status;
  int32_t* ret_prefix;
  int ret_prefix_stride;
};
struct RetainBatch {
  Geom g;
  RetainPair pr[kMaxMergePairs];  // blockIdx.z selects the pair
  int q4, dtype, chunks_per_seg, nseg, mode, do_retention, union_kv, region_rows, slack;
  float d_hint;  // fused prefill: raw layer-l rows exist only for tokens with d > d_hint (< 0: for all)
  double gamma;
};
__device__ __forceinline__ RetainParams retain_view(const RetainBatch& bp, int pair) {
  const RetainPair& r = bp.pr[pair];
  RetainParams p;
  p.g = bp.g;
#pragma unroll
  for (int i = 0; i < 2; ++i) {
    p.a_pool[i] = r.a_pool[i];
    p.c_pool[i] = r.c_pool[i];
    p.a_meta[i] = r.a_meta[i];
    p.c_meta[i] = r.c_meta[i];
    p.e_pool[i] = r.e_pool[i];
  }
  p.q4 = bp.q4;
  p.dtype = bp.dtype;
  p.dist = r.dist;
  p.seg_minmax = r.seg_minmax;
  p.chunk_count = r.chunk_count;
  p.chunk_offset = r.chunk_offset;
  p.chunk_eq = r.chunk_eq;
  p.seg_sel = r.seg_sel;
  p.ret_count = r.ret_count;
  p.ret_offset = r.ret_offset;
  p.ret_index = r.ret_index;
  p.ret_rows = r.ret_rows;
  p.ret_capacity = r.ret_capacity;
  p.status = r.status;
  p.ret_prefix = r.ret_prefix;
  p.ret_prefix_stride = r.ret_prefix_stride;
  p.chunks_per_seg = bp.chunks_per_seg;
  p.nseg = bp.nseg;
  p.mode = bp.mode;
  p.do_retention = bp.do_retention;
  p.union_kv = bp.union_kv;
  p.region_rows = bp.region_rows;
  p.slack = bp.slack;
  p.d_hint = bp.d_hint;
  p.gamma = bp.gamma;
  return p;
}

// Segment (tensor, b, h) number `ls` of the call's sequences [seq_begin, seq_begin + seq_count):
// ls = (tensor * seq_count + (b - seq_begin)) * H + h; returns its index in the pair's tables.
__device__ __forceinline__ int call_segment(const Geom& g, int ls, int& tensor, int& b, int& h) {
  h = ls % g.n_kv_heads;
  const int r = ls / g.n_kv_heads;
  b = g.seq_begin + r % g.seq_count;
  tensor = r / g.seq_count;
  return (tensor * g.batch + b) * g.n_kv_heads + h;
}

struct InitParams {
  Geom g;
  unsigned* seg_minmax[kMaxMergePairs];
  int32_t* status[kMaxMergePairs];
  int clear_status;  // a merge of the whole batch starts from clean status words; an admission keeps them
};
__global__ void merge_init_kernel(const __grid_constant__ InitParams ip) {
  grid_dep_wait();
  grid_dep_launch();
  const int i = blockIdx.x * blockDim.x + threadIdx.x;
  unsigned* seg_minmax = ip.seg_minmax[blockIdx.y];
  if (i < 2 * ip.g.seq_count * ip.g.n_kv_heads) {
    int tensor, b, h;
    const int seg = call_segment(ip.g, i, tensor, b, h);
    seg_minmax[2 * seg] = 0x7f800000u;
    seg_minmax[2 * seg + 1] = 0u;
  }
  if (ip.clear_status && i < MC_STATUS_WORDS) ip.status[blockIdx.y][i] = 0;
}

// The four consecutive distances starting at token tok0 (a multiple of 4: they lie in one page).
__device__ __forceinline__ float4 load_dist4(const RetainParams& p, int tensor, int b, int h, int tok0, bool& ok) {
  const int page = checked_page(p.g, b, tok0 >> p.g.page_shift, p.status);
  ok = page >= 0;
  if (!ok) return make_float4(0.f, 0.f, 0.f, 0.f);  // a page id outside the pools: its tokens are never kept
  return *reinterpret_cast<const float4*>(
      p.dist + (((size_t)page * p.g.n_kv_heads + h) * 2 + tensor) * p.g.page_size + (tok0 & (p.g.page_size - 1)));
}

// The retention passes give a chunk of 1024 tokens to one warp: lane l owns the 32 consecutive tokens
// [32 l, 32 l + 32) of the chunk, i.e. one or two pages' worth of distances (pages hold at least 16 tokens).
struct Dist32 {
  float4 d[8];
  unsigned ok;   // bit i: d[i] was loaded (its tokens exist and their page id is valid)
  int page[2];   // page of the lane's first and second 16 tokens (-1: none)
};
__device__ __forceinline__ void load_dist32(const RetainParams& p, int tensor, int b, int h, int tok0, int n, Dist32& r) {
  r.ok = 0u;
#pragma unroll
  for (int hf = 0; hf < 2; ++hf) {
    const int t = tok0 + 16 * hf;
    r.page[hf] = t < n ? checked_page(p.g, b, t >> p.g.page_shift, p.status) : -1;
  }
#pragma unroll
  for (int i = 0; i < 8; ++i) {
    const int t = tok0 + 4 * i;
    const int page = r.page[i >> 2];
    r.d[i] = make_float4(0.f, 0.f, 0.f, 0.f);
    if (t < n && page >= 0) {
      r.d[i] = *reinterpret_cast<const float4*>(
          p.dist + (((size_t)page * p.g.n_kv_heads + h) * 2 + tensor) * p.g.page_size + (t & (p.g.page_size - 1)));
      r.ok |= 1u << i;
    }
  }
}

// Eq. 4's decision as single-precision comparisons.  The rule is defined on the double-precision
// threshold thr formed from the fp32 extremes ((double)d > thr, or < thr as printed); for a binary32 d that
// is the same as d > round_down(thr) (d < round_up(thr)), and |d - thr| < 1e-6 is the same as
// round_down(thr - 1e-6) < d < round_up(thr + 1e-6).  Top-k reading: the k-th largest distance's bits
// decide (d >= 0, so unsigned order is float order).
struct KeepRule {
  int kind;  // 0: d > cmp, 1: d < cmp, 2: top-k
  float cmp, near_lo, near_hi;
  uint32_t v;
};
__device__ __forceinline__ KeepRule make_rule(const RetainParams& p, int seg) {
  KeepRule r;
  r.v = 0u;
  double thr;
  if (p.mode == MC_RETAIN_TOPK) {
    r.kind = 2;
    r.v = p.seg_sel[2 * seg];
    thr = (double)__uint_as_float(r.v);
    r.cmp = 0.f;
    if (r.v == 0xffffffffu) thr = -4.0;  // nothing is kept: nothing is near either (d lies in [0, 1])
  } else {
    const double lo = p.seg_minmax[2 * seg], hi = p.seg_minmax[2 * seg + 1];
    if (p.mode == MC_RETAIN_DISTINCT) {
      r.kind = 0;
      thr = hi - (hi - lo) * p.gamma;
      r.cmp = __double2float_rd(thr);
    } else {
      r.kind = 1;
      thr = lo + (hi - lo) * p.gamma;
      r.cmp = __double2float_ru(thr);
    }
  }
  r.near_lo = __double2float_rd(thr - 1e-6);
  r.near_hi = __double2float_ru(thr + 1e-6);
  return r;
}
// Masks over the lane's 32 tokens (bit 4 i + j = token tok0 + 4 i + j): `sure` = kept whatever the ties do,
// `eq` = kept only while the segment's quota of ties lasts (top-k reading: d equal to the k-th largest; ties
// go to lower indices).  `near` counts the tokens whose distance lies within 1e-6 of the decision
// threshold: the ones a different rounding of d could have decided the other way.
__device__ __forceinline__ void keep_masks32_one(const KeepRule& r, const Dist32& dd, int tok0, int n, unsigned& sure, unsigned& eq,
                                                 int* near) {
  sure = eq = 0u;
  unsigned nr = 0u;
  // (one loop per rule: the rule is the same for the whole launch, the loop bodies stay a few instructions per token)
  if (r.kind == 2) {
#pragma unroll
    for (int i = 0; i < 8; ++i) {
      const float d[4] = {dd.d[i].x, dd.d[i].y, dd.d[i].z, dd.d[i].w};
#pragma unroll
      for (int j = 0; j < 4; ++j) {
        const uint32_t key = __float_as_uint(d[j]);
        sure |= (key > r.v ? 1u : 0u) << (4 * i + j);
        eq |= (key == r.v ? 1u : 0u) << (4 * i + j);
      }
    }
  } else if (r.kind == 0) {
#pragma unroll
    for (int i = 0; i < 8; ++i) {
      const float d[4] = {dd.d[i].x, dd.d[i].y, dd.d[i].z, dd.d[i].w};
#pragma unroll
      for (int j = 0; j < 4; ++j) sure |= (d[j] > r.cmp ? 1u : 0u) << (4 * i + j);
    }
  } else {
#pragma unroll
    for (int i = 0; i < 8; ++i) {
      const float d[4] = {dd.d[i].x, dd.d[i].y, dd.d[i].z, dd.d[i].w};
#pragma unroll
      for (int j = 0; j < 4; ++j) sure |= (d[j] < r.cmp ? 1u : 0u) << (4 * i + j);
    }
  }
  // tokens that exist (before the sequence's end, in a page with a valid id)
  unsigned valid = 0u;
#pragma unroll
  for (int i = 0; i < 8; ++i)
    if (dd.ok & (1u << i)) valid |= 0xFu << (4 * i);
  const int left = n - tok0;
  valid &= left >= 32 ? 0xffffffffu : (left > 0 ? (1u << left) - 1u : 0u);
  sure &= valid;
  eq &= valid;
  if (near) {
#pragma unroll
    for (int i = 0; i < 8; ++i) {
      const float d[4] = {dd.d[i].x, dd.d[i].y, dd.d[i].z, dd.d[i].w};
#pragma unroll
      for (int j = 0; j < 4; ++j) nr |= (d[j] > r.near_lo && d[j] < r.near_hi ? 1u : 0u) << (4 * i + j);
    }
    *near += __popc(nr & valid);
  }
}

// The decision for the lane's 32 tokens of segment (tensor, b, h), distances included.  With one set for keys
// and values (union_kv; threshold modes only) the other tensor's rule is applied to its own distances as
// well and the two masks are joined; `near` counts this tensor's own near-threshold tokens either way.
// `page` receives the pages of the lane's first and second 16 tokens.
__device__ __forceinline__ void keep_masks32(const RetainParams& p, int seg, int tensor, int b, int h, int tok0, int n,
                                             unsigned& sure, unsigned& eq, int (&page)[2], int* near = nullptr) {
  Dist32 dd;
  load_dist32(p, tensor, b, h, tok0, n, dd);
  page[0] = dd.page[0];
  page[1] = dd.page[1];
  keep_masks32_one(make_rule(p, seg), dd, tok0, n, sure, eq, near);
  if (p.union_kv && p.mode != MC_RETAIN_TOPK) {
    const int seg_o = tensor ? seg - p.g.batch * p.g.n_kv_heads : seg + p.g.batch * p.g.n_kv_heads;
    unsigned sure_o, eq_o;
    load_dist32(p, 1 - tensor, b, h, tok0, n, dd);
    keep_masks32_one(make_rule(p, seg_o), dd, tok0, n, sure_o, eq_o, nullptr);
    sure |= sure_o;
  }
}

// Top-k reading of the retention rule: per segment, the k-th largest distance (k = ceil(gamma n)) by a
// radix select over the float bits (d >= 0, so unsigned order is float order), and how many of the
// tokens equal to it belong to the k largest.
__global__ void __launch_bounds__(kRetThreads) retain_select_kernel(const __grid_constant__ RetainBatch bp) {
  grid_dep_wait();
  grid_dep_launch();
  const RetainParams p = retain_view(bp, blockIdx.z);
  __shared__ int hist[256];
  __shared__ uint32_t s_prefix, s_mask;
  __shared__ int s_remaining;
  int tensor, b, h;
  const int seg = call_segment(p.g, blockIdx.x, tensor, b, h);
  const int n = checked_len(p.g, b, p.status);
  const int k = min(n, (int)ceil(p.gamma * (double)n - 1e-12));
  if (k <= 0 || !p.do_retention) {
    if (threadIdx.x == 0) {
      p.seg_sel[2 * seg] = 0xffffffffu;  // nothing is larger, nothing is equal
      p.seg_sel[2 * seg + 1] = 0u;
    }
    return;
  }
  if (threadIdx.x == 0) {
    s_prefix = 0u;
    s_mask = 0u;
    s_remaining = k;
  }
  for (int pass = 0; pass < 4; ++pass) {
    const int shift = 24 - 8 * pass;
    hist[threadIdx.x] = 0;
    __syncthreads();
    const uint32_t prefix = s_prefix, mask = s_mask;
    for (int tok0 = 4 * threadIdx.x; tok0 < n; tok0 += 4 * kRetThreads) {
      bool ok;
      const float4 d4 = load_dist4(p, tensor, b, h, tok0, ok);
      const float d[4] = {d4.x, d4.y, d4.z, d4.w};
#pragma unroll
      for (int j = 0; j < 4; ++j) {
        const uint32_t key = __float_as_uint(d[j]);
        if (tok0 + j < n && (key & mask) == prefix) atomicAdd(&hist[(key >> shift) & 255u], 1);
      }
    }
    __syncthreads();
    if (threadIdx.x == 0) {
      int remaining = s_remaining, bin = 255;
      for (; bin > 0; --bin) {  // from the largest digit down: the bin holding the `remaining`-th largest key
        if (hist[bin] >= remaining) break;
        remaining -= hist[bin];
      }
      s_remaining = remaining;
      s_prefix = prefix | ((uint32_t)bin << shift);
      s_mask = mask | (255u << shift);
    }
    __syncthreads();
  }
  if (threadIdx.x == 0) {
    p.seg_sel[2 * seg] = s_prefix;                  // the k-th largest distance
    p.seg_sel[2 * seg + 1] = (uint32_t)s_remaining;  // of the tokens equal to it, this many (the lowest indices) are kept
  }
}

// Per (segment, 1024-token chunk): how many tokens Eq. 4 keeps; one warp per chunk (a lane looks at 32
// consecutive tokens), eight chunks per block in (segment, chunk) order.  The block that finishes last
// (ticket in a status word) turns the counts into offsets: exclusive scan in (segment, chunk) order.
__global__ void __launch_bounds__(kRetThreads) retain_count_kernel(const __grid_constant__ RetainBatch bp) {
  grid_dep_wait();
  grid_dep_launch();
  const RetainParams p = retain_view(bp, blockIdx.z);
  __shared__ int s_cnt[kRetThreads / 32];
  __shared__ int s_last;
  __shared__ int s_carry;
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  const int n_items = 2 * p.g.seq_count * p.g.n_kv_heads * p.chunks_per_seg;
  const int item = blockIdx.x * (kRetThreads / 32) + warp;
  if (item < n_items) {  // (warp-uniform)
    const int chunk = item % p.chunks_per_seg;
    int tensor, b, h;
    const int seg = call_segment(p.g, item / p.chunks_per_seg, tensor, b, h);
    const int n = checked_len(p.g, b, p.status);
    int cnt = 0, cnt_eq = 0, cnt_near = 0;
    if (p.do_retention && chunk * kChunk < n) {
      unsigned sure, eq;
      int page[2];
      keep_masks32(p, seg, tensor, b, h, chunk * kChunk + 32 * lane, n, sure, eq, page, &cnt_near);
      cnt = __popc(sure);
      cnt_eq = __popc(eq);
    }
    for (int o = 16; o; o >>= 1) {
      cnt += __shfl_xor_sync(0xffffffffu, cnt, o);
      cnt_eq += __shfl_xor_sync(0xffffffffu, cnt_eq, o);
      cnt_near += __shfl_xor_sync(0xffffffffu, cnt_near, o);
    }
    if (lane == 0) {
      p.chunk_count[(size_t)seg * p.chunks_per_seg + chunk] = cnt;
      p.chunk_eq[(size_t)seg * p.chunks_per_seg + chunk] = cnt_eq;
      if (cnt_near) atomicAdd(&p.status[MC_STATUS_NEAR_THRESHOLD], cnt_near);
      if (chunk == 0 && p.do_retention && p.d_hint >= 0.f && n > 0 && p.mode == MC_RETAIN_DISTINCT) {
        // fused prefill: every token this segment keeps must be one whose raw row was stored (d > d_hint)
        const double lo = p.seg_minmax[2 * seg], hi = p.seg_minmax[2 * seg + 1];
        if (hi - (hi - lo) * p.gamma < (double)p.d_hint && hi > lo && p.gamma > 0.0) atomicOr(&p.status[MC_STATUS_FLAGS], MC_FLAG_HINT_TOO_HIGH);
      }
      __threadfence();  // the counts, before this block's ticket
    }
  }
  __syncthreads();
  if (threadIdx.x == 0) {
    __threadfence();
    const int ticket = atomicAdd(&p.status[MC_STATUS_RESERVED1], 1);
    s_last = ticket == (int)gridDim.x - 1;
    s_carry = 0;
  }
  __syncthreads();
  if (!s_last) return;
  __threadfence();
  // ---- last block.  Top-k mode first: the ties are handed out in token order, so per segment the
  // chunks take from the quota one after the other; chunk_eq becomes "ties before this chunk".
  if (p.mode == MC_RETAIN_TOPK) {
    for (int ls = threadIdx.x; ls < 2 * p.g.seq_count * p.g.n_kv_heads; ls += kRetThreads) {
      int t_, b_, h_;
      const int sg = call_segment(p.g, ls, t_, b_, h_);
      const int quota = (int)p.seg_sel[2 * sg + 1];
      int eq_run = 0;
      for (int c = 0; c < p.chunks_per_seg; ++c) {
        const size_t ci = (size_t)sg * p.chunks_per_seg + c;
        const int e = __ldcg(p.chunk_eq + ci);
        p.chunk_count[ci] = __ldcg(p.chunk_count + ci) + max(0, min(e, quota - eq_run));
        p.chunk_eq[ci] = eq_run;
        eq_run += e;
      }
    }
    __threadfence();
    __syncthreads();
  }
  if (p.region_rows > 0) {
    // ---- admission: every sequence of the call owns the entries [b R, (b + 1) R) of the pool, its
    // segments in (tensor, head) order inside them.  A sequence that needs more keeps nothing
    // (offset -1) and the overflow flag is set.
    const int per_seq = 2 * p.g.n_kv_heads * p.chunks_per_seg;
    for (int sq = 0; sq < p.g.seq_count; ++sq) {
      const int bq = p.g.seq_begin + sq;
      __syncthreads();
      if (threadIdx.x == 0) s_carry = 0;
      __syncthreads();
      for (int base = 0; base < per_seq; base += kRetThreads) {
        const int j = base + threadIdx.x;  // (tensor, head, chunk), chunk fastest
        const int sg = j < per_seq ? ((j / p.chunks_per_seg / p.g.n_kv_heads) * p.g.batch + bq) * p.g.n_kv_heads +
                                         (j / p.chunks_per_seg) % p.g.n_kv_heads : 0;
        const size_t ci = (size_t)sg * p.chunks_per_seg + (j % p.chunks_per_seg);
        // (the free entries of a segment follow its last chunk's)
        const int v = j < per_seq ? __ldcg(p.chunk_count + ci) + (j % p.chunks_per_seg == p.chunks_per_seg - 1 ? p.slack : 0) : 0;
        int x = v;
        for (int o = 1; o < 32; o <<= 1) {
          const int y = __shfl_up_sync(0xffffffffu, x, o);
          if (lane >= o) x += y;
        }
        if (lane == 31) s_cnt[warp] = x;
        __syncthreads();
        int warp_excl = 0;
        for (int w = 0; w < warp; ++w) warp_excl += s_cnt[w];
        const int excl = s_carry + warp_excl + x - v;
        if (j < per_seq) p.chunk_offset[ci] = bq * p.region_rows + excl;
        __syncthreads();
        if (threadIdx.x == kRetThreads - 1) s_carry = excl + v;
        __syncthreads();
      }
      const bool fits = s_carry <= p.region_rows;
      for (int sj = threadIdx.x; sj < 2 * p.g.n_kv_heads; sj += kRetThreads) {
        const int sg = ((sj / p.g.n_kv_heads) * p.g.batch + bq) * p.g.n_kv_heads + sj % p.g.n_kv_heads;
        int cnt_seg = 0;
        for (int c = 0; c < p.chunks_per_seg; ++c) cnt_seg += __ldcg(p.chunk_count + (size_t)sg * p.chunks_per_seg + c);
        p.ret_offset[sg] = fits ? p.chunk_offset[(size_t)sg * p.chunks_per_seg] : -1;
        p.ret_count[sg] = fits ? cnt_seg : 0;
      }
      if (threadIdx.x == 0 && !fits) atomicOr(&p.status[MC_STATUS_FLAGS], MC_FLAG_RETAIN_OVERFLOW);
    }
    if (threadIdx.x == 0) p.status[MC_STATUS_RESERVED1] = 0;
    return;
  }
  // exclusive scan of all chunk counts
  const int total = p.nseg * p.chunks_per_seg;
  for (int base = 0; base < total; base += kRetThreads) {
    const int i = base + threadIdx.x;
    const int v = i < total ? __ldcg(p.chunk_count + i) + (i % p.chunks_per_seg == p.chunks_per_seg - 1 ? p.slack : 0) : 0;
    int x = v;
    for (int o = 1; o < 32; o <<= 1) {
      const int y = __shfl_up_sync(0xffffffffu, x, o);
      if (lane >= o) x += y;
    }
    if (lane == 31) s_cnt[warp] = x;
    __syncthreads();
    int warp_excl = 0;
    for (int w = 0; w < warp; ++w) warp_excl += s_cnt[w];
    const int excl = s_carry + warp_excl + x - v;
    if (i < total) {
      p.chunk_offset[i] = excl;
      if (i % p.chunks_per_seg == 0) p.ret_offset[i / p.chunks_per_seg] = excl;
    }
    __syncthreads();
    if (threadIdx.x == kRetThreads - 1) s_carry = excl + v;
    __syncthreads();
  }
  if (threadIdx.x == 0) {
    const int sum = s_carry;
    p.ret_offset[p.nseg] = sum;
    p.status[MC_STATUS_RETAINED_TOTAL] = sum - p.nseg * p.slack;
    p.status[MC_STATUS_RESERVED1] = 0;
    if ((int64_t)sum > p.ret_capacity) atomicOr(&p.status[MC_STATUS_FLAGS], MC_FLAG_RETAIN_OVERFLOW);
  }
}

// Per (segment, chunk), one warp each: ordered compaction of the kept token indices, their scales zeroed,
// bit copies of both layers' rows, and the chunk's eight entries of the prefix table (one per 128 tokens =
// four lanes).  Writes ret_count per segment.
__global__ void __launch_bounds__(kRetThreads) retain_compact_kernel(const __grid_constant__ RetainBatch bp) {
  grid_dep_wait();
  grid_dep_launch();
  const RetainParams p = retain_view(bp, blockIdx.z);
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  const int n_items = 2 * p.g.seq_count * p.g.n_kv_heads * p.chunks_per_seg;
  const int item = blockIdx.x * (kRetThreads / 32) + warp;
  if (item >= n_items) return;  // (no block-wide barrier below)
  const int chunk = item % p.chunks_per_seg;
  int tensor, b, h;
  const int seg = call_segment(p.g, item / p.chunks_per_seg, tensor, b, h);
  const int n = checked_len(p.g, b, p.status);
  const int seg_off = p.ret_offset[seg];
  // (admission: the scan has written the segment's count, and -1 as the offset of a sequence that did not fit)
  const bool overflow = p.region_rows > 0 ? seg_off < 0 : (int64_t)p.ret_offset[p.nseg] > p.ret_capacity;
  const int seg_cnt = overflow ? 0 : (p.region_rows > 0 ? p.ret_count[seg] : p.ret_offset[seg + 1] - seg_off - p.slack);
  int32_t* prefix = p.ret_prefix + (size_t)seg * p.ret_prefix_stride;
  if (chunk == 0) {
    __syncwarp();  // (every lane has read ret_count)
    if (lane == 0) p.ret_count[seg] = seg_cnt;
    if (!overflow)  // the free entries behind the list
      for (int j = lane; j < p.slack; j += 32) {
        const int64_t pos = (int64_t)seg_off + seg_cnt + j;
        if (MC_IN_BOUNDS(pos >= 0 && pos < p.ret_capacity, p.status)) p.ret_index[pos] = -1;
      }
    // table entries past the last chunk: everything lies before them
    for (int j = p.chunks_per_seg * (kChunk / 128) + lane; j < p.ret_prefix_stride; j += 32) prefix[j] = seg_cnt;
  }
  const int pj = chunk * (kChunk / 128) + (lane >> 2);  // the table entry of the lane's 128 tokens
  const bool active = !overflow && p.do_retention && chunk * kChunk < n;
  if (!active) {
    if ((lane & 3) == 0 && pj < p.ret_prefix_stride) prefix[pj] = seg_cnt;  // chunk past the sequence (or nothing retained)
    return;
  }
  const size_t ci = (size_t)seg * p.chunks_per_seg + chunk;
  const int my_count = p.chunk_count[ci];
  const int out0 = p.chunk_offset[ci];
  const int tok0 = chunk * kChunk + 32 * lane;
  unsigned m, m_eq;
  int page[2];
  keep_masks32(p, seg, tensor, b, h, tok0, n, m, m_eq, page);
  if (p.mode == MC_RETAIN_TOPK) {
    // ties: kept while the segment's quota lasts, in token order (ordered count of the ties before each)
    const int ce = __popc(m_eq);
    int xe = ce;
    for (int o = 1; o < 32; o <<= 1) {
      const int y = __shfl_up_sync(0xffffffffu, xe, o);
      if (lane >= o) xe += y;
    }
    int seen = p.chunk_eq[ci] + xe - ce;
    const int quota = (int)p.seg_sel[2 * seg + 1];
    for (unsigned rest = m_eq; rest; rest &= rest - 1) {
      if (seen < quota) m |= rest & (0u - rest);
      ++seen;
    }
  }
  const int c = __popc(m);
  int x = c;
  for (int o = 1; o < 32; o <<= 1) {
    const int y = __shfl_up_sync(0xffffffffu, x, o);
    if (lane >= o) x += y;
  }
  if ((lane & 3) == 0 && pj < p.ret_prefix_stride) prefix[pj] = out0 - seg_off + x - c;
  int pos = out0 + x - c;
  for (unsigned rest = m; rest; rest &= rest - 1) {  // (kept tokens lie in a page that keep_masks32 has checked)
    const int j = __ffs(rest) - 1;
    const int tok = tok0 + j;
    float* sc = reinterpret_cast<float*>((tensor ? p.e_pool[1] : p.e_pool[0]) + ((size_t)((j >> 4) ? page[1] : page[0]) * p.g.n_kv_heads + h) * tile_bytes(p.g.page_size) +
                                         p.g.page_size * kRowBytes) + (tok & (p.g.page_size - 1));
    if (!MC_IN_BOUNDS(pos >= 0 && pos < p.ret_capacity, p.status)) continue;  // (range-checked build)
    p.ret_index[pos++] = tok;
    // a retained token is served from its raw rows: the scale -0 makes the shared direction
    // contribute nothing for it wherever scales are applied blindly, and tells the attention
    // kernel that the token's score comes from its raw key row
    sc[0] = -0.f;
    sc[p.g.page_size] = -0.f;
  }
  // gather: the warp copies both layers' raw rows of one entry at a time (a half-warp per layer), four
  // entries in flight.  Which token an entry is comes from the lane that kept it (its mask and its pages),
  // not from memory: the copies of different entries do not wait on one another.
  const int layer = lane >> 4, l16 = lane & 15;
  const int excl = x - c;
  const char* pool = layer ? (tensor ? p.c_pool[1] : p.c_pool[0]) : (tensor ? p.a_pool[1] : p.a_pool[0]);
  for (int e0 = 0; e0 < my_count; e0 += 4) {
    int tok_u[4];
    size_t row_u[4];
#pragma unroll
    for (int u = 0; u < 4; ++u) {
      const int e = e0 + u;
      const bool mine = e >= excl && e < excl + c;
      const unsigned own = __ballot_sync(0xffffffffu, mine);
      const int src = own ? __ffs(own) - 1 : 0;
      const int j = __shfl_sync(0xffffffffu, mine ? (int)__fns(m, 0, e - excl + 1) : 0, src);
      const int pg0 = __shfl_sync(0xffffffffu, page[0], src), pg1 = __shfl_sync(0xffffffffu, page[1], src);
      const int tok = chunk * kChunk + 32 * src + j;
      const int pg = (j >> 4) ? pg1 : pg0;
      // (an entry past the lanes' kept tokens, or past the pool in the range-checked build, is skipped)
      const bool ok = own != 0u && e < my_count && pg >= 0 && MC_IN_BOUNDS(out0 >= 0 && (int64_t)out0 + e < p.ret_capacity, p.status);
      tok_u[u] = ok ? tok : -1;
      row_u[u] = ((size_t)max(pg, 0) * p.g.n_kv_heads + h) * p.g.page_size + (tok & (p.g.page_size - 1));
    }
    if (!p.q4) {
      uint4 v[4];
#pragma unroll
      for (int u = 0; u < 4; ++u)
        if (tok_u[u] >= 0) v[u] = *reinterpret_cast<const uint4*>(pool + row_u[u] * kRowBytes + l16 * 16);
#pragma unroll
      for (int u = 0; u < 4; ++u)
        if (tok_u[u] >= 0) {
          char* dst = p.ret_rows + ((size_t)layer * p.ret_capacity + out0 + e0 + u) * kRetEntryBytes;
          *reinterpret_cast<uint4*>(dst + l16 * 16) = v[u];
          if (l16 == 0) *reinterpret_cast<int4*>(dst + kRowBytes) = make_int4(tok_u[u], 0, 0, 0);
        }
      continue;
    }
#pragma unroll
    for (int u = 0; u < 4; ++u) {
      if (tok_u[u] < 0) continue;
      const size_t row = row_u[u];
      char* dst = p.ret_rows + ((size_t)layer * p.ret_capacity + out0 + e0 + u) * kRetEntryBytes;
      // lane l16: channels [8 l16, 8 l16 + 8).  code * scale + zero is formed in double (exact) and
      // rounded once to the storage type, so the row is the same bits on any machine.
      const char* codes = pool + row * kQ4RowBytes;
      const char* meta = layer ? (tensor ? p.c_meta[1] : p.c_meta[0]) : (tensor ? p.a_meta[1] : p.a_meta[0]);
      const uint32_t w = *reinterpret_cast<const uint32_t*>(codes + l16 * 4);
      const __half2* mp = tensor == 0 ? reinterpret_cast<const __half2*>(meta) + (row / p.g.page_size) * 128 + 8 * l16
                                      : reinterpret_cast<const __half2*>(meta) + row * 4 + (l16 >> 2);
      uint32_t o[4];
#pragma unroll
      for (int j = 0; j < 4; ++j) {
        unsigned short hb[2];
#pragma unroll
        for (int q = 0; q < 2; ++q) {
          const int ch = 2 * j + q;
          const __half2 sz = tensor == 0 ? mp[ch] : mp[0];
          const double v = (double)((w >> (4 * ch)) & 15u) * (double)__low2float(sz) + (double)__high2float(sz);
          if (p.dtype == MC_F16) {
            const __half hv = __double2half(v);
            hb[q] = *reinterpret_cast<const unsigned short*>(&hv);
          } else {
            const __nv_bfloat16 bv = __double2bfloat16(v);
            hb[q] = *reinterpret_cast<const unsigned short*>(&bv);
          }
        }
        o[j] = (uint32_t)hb[0] | ((uint32_t)hb[1] << 16);
      }
      *reinterpret_cast<uint4*>(dst + l16 * 16) = make_uint4(o[0], o[1], o[2], o[3]);
      if (l16 == 0) *reinterpret_cast<int4*>(dst + kRowBytes) = make_int4(tok_u[u], 0, 0, 0);
    }
  }
}

// ---------------------------------------------------------------------------------------------
// Decode-time append (Algorithm 2 "MiniCache Decoding": merge of the new token pair)
// ---------------------------------------------------------------------------------------------
template <int DT>
__global__ void __launch_bounds__(128) append_kernel(const AppendParams p) {
  grid_dep_launch();
  append_row<DT>(p, blockIdx.x * (128 / 16) + (threadIdx.x >> 4), threadIdx.x & 15, [] { grid_dep_wait(); });
}

// ---------------------------------------------------------------------------------------------
// Host launchers
// ---------------------------------------------------------------------------------------------
static inline int chunks_per_seg(int max_seq_len) { return max_seq_len > 0 ? (max_seq_len + kChunk - 1) / kChunk : 1; }

size_t merge_workspace_bytes(const mc_config* cfg, const mc_batch* bt) {
  const size_t nseg = (size_t)2 * bt->batch * cfg->n_kv_heads;
  return align_up(nseg * chunks_per_seg(bt->max_seq_len) * sizeof(int32_t), 256) * 3 + align_up(nseg * 2 * sizeof(uint32_t), 256);
}

mc_status launch_merge_pairs(const mc_config* cfg, const mc_batch* bt, const Geom& g, int n_pairs, const mc_layer_kv* const* lm1,
                             const mc_layer_kv* const* l, const mc_layer_q4* const* q_lm1, const mc_layer_q4* const* q_l,
                             const mc_pair_cache* const* out, int do_retention, void* workspace, cudaStream_t stream,
                             int region_rows, const PrefillHook* hook) {
  const bool q4 = q_lm1 != nullptr;
  if (hook != nullptr && (n_pairs != 1 || q4)) return MC_ERR_UNSUPPORTED;
  const int nseg = 2 * bt->batch * cfg->n_kv_heads;
  const int nseg_call = 2 * g.seq_count * cfg->n_kv_heads;  // segments of the sequences this call works on
  // every shape limit before the first launch
  if (n_pairs < 1 || n_pairs > kMaxMergePairs) return MC_ERR_SHAPE;
  if (bt->batch > kMergeMaxBatchSmem) return MC_ERR_SHAPE;  // the sequences' page prefix lives in shared memory
  if (2LL * n_pairs * bt->batch * ((bt->max_seq_len + cfg->page_size - 1) / cfg->page_size) *
          ((cfg->n_kv_heads * cfg->page_size + kRowsPerItem - 1) / kRowsPerItem) > 0x7fffffffLL)
    return MC_ERR_SHAPE;
  InitParams ip;
  for (int i = 0; i < kMaxMergePairs; ++i) {
    ip.seg_minmax[i] = reinterpret_cast<unsigned*>(out[std::min(i, n_pairs - 1)]->seg_minmax);
    ip.status[i] = out[std::min(i, n_pairs - 1)]->status;
  }
  ip.g = g;
  ip.clear_status = region_rows > 0 ? 0 : 1;
  MC_CUDA_CHECK(launch_pdl(merge_init_kernel, dim3((std::max(nseg_call, (int)MC_STATUS_WORDS) + 255) / 256, n_pairs), dim3(256), 0, stream, ip));
  MC_CUDA_CHECK(cudaGetLastError());
  if (bt->batch == 0 || g.seq_count == 0) return MC_OK;

  MergeParams mp;
  RetainBatch rb;
  mp.g = g;
  rb.g = g;
  const size_t arr = align_up((size_t)nseg * chunks_per_seg(bt->max_seq_len) * sizeof(int32_t), 256);
  const size_t ws_pair = merge_workspace_bytes(cfg, bt);
  for (int i = 0; i < kMaxMergePairs; ++i) {
    const int j = std::min(i, n_pairs - 1);  // (unused slots repeat the last pair: no null pointers in the parameters)
    MergePair& m = mp.pr[i];
    m.a_pool[0] = (const char*)(q4 ? q_lm1[j]->k_codes : lm1[j]->k_pool);
    m.a_pool[1] = (const char*)(q4 ? q_lm1[j]->v_codes : lm1[j]->v_pool);
    m.c_pool[0] = (const char*)(q4 ? q_l[j]->k_codes : l[j]->k_pool);
    m.c_pool[1] = (const char*)(q4 ? q_l[j]->v_codes : l[j]->v_pool);
    m.a_meta[0] = (const char*)(q4 ? q_lm1[j]->k_meta : nullptr);
    m.a_meta[1] = (const char*)(q4 ? q_lm1[j]->v_meta : nullptr);
    m.c_meta[0] = (const char*)(q4 ? q_l[j]->k_meta : nullptr);
    m.c_meta[1] = (const char*)(q4 ? q_l[j]->v_meta : nullptr);
    m.e_pool[0] = (char*)out[j]->e_k;
    m.e_pool[1] = (char*)out[j]->e_v;
    m.dist = out[j]->dist;
    m.seg_minmax = reinterpret_cast<unsigned*>(out[j]->seg_minmax);
    m.status = out[j]->status;
    RetainPair& r = rb.pr[i];
    for (int t = 0; t < 2; ++t) {
      r.a_pool[t] = m.a_pool[t];
      r.c_pool[t] = m.c_pool[t];
      r.a_meta[t] = m.a_meta[t];
      r.c_meta[t] = m.c_meta[t];
      r.e_pool[t] = m.e_pool[t];
    }
    r.dist = out[j]->dist;
    r.seg_minmax = out[j]->seg_minmax;
    char* ws = (char*)workspace + (size_t)j * ws_pair;
    r.chunk_count = reinterpret_cast<int32_t*>(ws);
    r.chunk_offset = reinterpret_cast<int32_t*>(ws + arr);
    r.chunk_eq = reinterpret_cast<int32_t*>(ws + 2 * arr);
    r.seg_sel = reinterpret_cast<uint32_t*>(ws + 3 * arr);
    r.ret_count = out[j]->ret_count;
    r.ret_offset = out[j]->ret_offset;
    r.ret_index = out[j]->ret_index;
    r.ret_rows = (char*)out[j]->ret_rows;
    r.ret_capacity = out[j]->ret_capacity;
    r.status = out[j]->status;
    r.ret_prefix = out[j]->ret_prefix;
    r.ret_prefix_stride = (int)out[j]->ret_prefix_stride;
  }
  mp.n_pairs = n_pairs;
  mp.merge_fn = cfg->merge_fn;
  mp.t_mode = cfg->t_mode;
  mp.ta = (float)(1.0 - cfg->t);
  mp.tc = (float)cfg->t;
  mp.items_per_page = (cfg->n_kv_heads * cfg->page_size + kRowsPerItem - 1) / kRowsPerItem;
  // upper bound of the item count (the kernel enumerates the pages that hold tokens)
  const long long total = 2LL * n_pairs * g.seq_count * ((bt->max_seq_len + cfg->page_size - 1) / cfg->page_size) * mp.items_per_page;
  if (hook != nullptr) {
    if (mc_status st = launch_prefill_merge(cfg, bt, g, hook->proj, lm1[0], l[0], out[0], hook->d_hint, stream)) return st;
  } else if (total > 0) {
    int n_sm = 0;
    if (mc_status st = sm_count(&n_sm)) return st;
    const int grid = (int)std::min<long long>((long long)n_sm * kMergeCtasPerSm, total);
    const size_t smem = 128 + (size_t)kMergeStages * kMergeStageBytes + (kMergeStages + 2 * kMergeMaxBatchSmem + 3) * 4 + 8 +
                        2 * kMergeStages * 8 + 64;
    void (*kern)(const MergeParams) =
        cfg->dtype == MC_F16 ? (q4 ? merge_kernel<MC_F16, true> : merge_kernel<MC_F16, false>)
                             : (q4 ? merge_kernel<MC_BF16, true> : merge_kernel<MC_BF16, false>);
    MC_CUDA_CHECK(cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem));
    MC_CUDA_CHECK(launch_pdl(kern, dim3(grid), dim3(kMergeThreads), smem, stream, mp));
  }

  rb.q4 = q4 ? 1 : 0;
  rb.dtype = cfg->dtype;
  rb.chunks_per_seg = chunks_per_seg(bt->max_seq_len);
  rb.nseg = nseg;
  rb.mode = cfg->retain_mode;
  rb.do_retention = do_retention;
  rb.union_kv = cfg->retain_union;
  rb.region_rows = region_rows;
  rb.slack = cfg->append_slack;
  rb.d_hint = hook != nullptr ? hook->d_hint : -1.f;
  rb.gamma = cfg->gamma;
  dim3 grid((rb.chunks_per_seg * nseg_call + kRetThreads / 32 - 1) / (kRetThreads / 32), 1, n_pairs);  // a warp per (segment, chunk)
  if (cfg->retain_mode == MC_RETAIN_TOPK)
    MC_CUDA_CHECK(launch_pdl(retain_select_kernel, dim3(nseg_call, 1, n_pairs), dim3(kRetThreads), 0, stream, rb));
  MC_CUDA_CHECK(launch_pdl(retain_count_kernel, dim3(grid), dim3(kRetThreads), 0, stream, rb));
  MC_CUDA_CHECK(launch_pdl(retain_compact_kernel, dim3(grid), dim3(kRetThreads), 0, stream, rb));
  return MC_OK;
}

mc_status launch_merge(const mc_config* cfg, const mc_batch* bt, const Geom& g, const mc_layer_kv* lm1,
                       const mc_layer_kv* l, const mc_layer_q4* q_lm1, const mc_layer_q4* q_l, const mc_pair_cache* out,
                       int do_retention, void* workspace, cudaStream_t stream) {
  return launch_merge_pairs(cfg, bt, g, 1, lm1 ? &lm1 : nullptr, l ? &l : nullptr, q_lm1 ? &q_lm1 : nullptr, q_l ? &q_l : nullptr,
                            &out, do_retention, workspace, stream, 0);
}

mc_status launch_append(const mc_config* cfg, const mc_batch* bt, const Geom& g, const mc_pair_cache* pair,
                        const void* k_new_lm1, const void* v_new_lm1, const void* k_new_l, const void* v_new_l,
                        cudaStream_t stream) {
  const AppendParams ap = make_append_params(cfg, bt, g, pair, k_new_lm1, v_new_lm1, k_new_l, v_new_l);
  if (ap.total_rows == 0) return MC_OK;
  const int blocks = (ap.total_rows + 7) / 8;
  if (cfg->dtype == MC_F16)
    MC_CUDA_CHECK(launch_pdl(append_kernel<MC_F16>, dim3(blocks), dim3(128), 0, stream, ap));
  else
    MC_CUDA_CHECK(launch_pdl(append_kernel<MC_BF16>, dim3(blocks), dim3(128), 0, stream, ap));
  MC_CUDA_CHECK(cudaGetLastError());
  return MC_OK;
}

}  // namespace mc
