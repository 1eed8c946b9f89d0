// Merge fused into the prefill (Algorithm 1: "merge at odd layers during prefill, then delete layer l-1"):
// layer l's keys / values are produced on chip by their projection K^l = X W_k^T (V alike) and merged with
// layer l-1's cached rows (Eq. 2, Eq. 3, distance of Sec. 4.2) in the projection's epilogue, so the rows of
// layer l never travel to HBM and back; only the rows of tokens whose distance exceeds a hint are stored
// raw, for the retention rule (Eq. 4) to pick from afterwards.
//
// One CTA = one tile of 128 tokens x the 128 channels of one (tensor, kv head):
//   warp 0      streams X and W tiles (128 x 64 each, 16-bit, 128-byte swizzle) through a ring of
//               shared-memory stages with tensor-map bulk copies (TMA)
//   warp 1      owns the tensor memory (128 columns x 128 lanes of fp32 accumulators) and issues the
//               5th-generation tensor-core instructions (tcgen05.mma, operands straight from shared memory)
//   warps 2..5  epilogue: a thread takes one token row out of tensor memory (its 128 channels), rounds it
//               to the storage type -- these are layer l's rows --, fetches layer l-1's row, merges, and
//               writes the shared direction, the scales and the distance in the pair cache's tile format
// Two CTAs share an SM (two ring stages of 32 KB and the epilogue's row staging each, 128 of the 512 tensor-memory
// columns, under 100 registers per thread): while one is in its epilogue the other's main loop has the tensor
// cores and the copy engine.
// Every wait is bounded; tensor memory is released on every path.
#include <cuda.h>

#include <algorithm>
#include <mutex>

#include "mc_common.cuh"
#include "mc_kernels.h"
#include "mc_pipe.cuh"

namespace mc {

constexpr int kPfTileM = 128;   // tokens per tile
constexpr int kPfTileN = 128;   // channels per tile = one head
constexpr int kPfTileK = 64;    // elements per stage row: 128 bytes, the swizzle span
constexpr int kPfStages = 2;
constexpr int kPfStageBytes = (kPfTileM + kPfTileN) * kPfTileK * 2;  // X tile, then W tile of one head: 32 KB
constexpr int kPfThreads = 192;
constexpr int kPfTmemCols = 128;  // per head
constexpr int kPfEpiRow = kRowBytes + 16;           // a staged row, padded: 32 rows fall into different banks
constexpr int kPfEpiWarp = 32 * kPfEpiRow;          // staging of one epilogue warp's 32 rows: 8704 bytes

struct PrefillParams {
  Geom g;
  const char* a_pool[2];  // layer l-1: K, V pools
  char* c_pool[2];        // layer l: K, V pools; rows of tokens with d > d_hint are stored here
  char* e_pool[2];
  float* dist;
  unsigned* seg_minmax;
  int32_t* status;
  int x_seq_stride;  // rows of X per sequence (a multiple of 128)
  int d_model;
  int n_mtiles;      // token tiles in all: batch * x_seq_stride / 128
  int mt_group, ht_group, n_htg;  // tile order, see below
  int n_hgroups;  // columns per tensor: kv heads / heads per CTA
  float ta, tc;
  int t_mode;
  float d_hint;
};

// ---- PTX wrappers of this file ------------------------------------------------------------------
__device__ __forceinline__ void tma_load_2d(uint32_t dst, const CUtensorMap* map, int x, int y, uint32_t bar) {
  asm volatile("cp.async.bulk.tensor.2d.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%2, %3}], [%4];" ::"r"(dst),
               "l"(reinterpret_cast<uint64_t>(map)), "r"(x), "r"(y), "r"(bar)
               : "memory");
}
__device__ __forceinline__ void tmem_alloc(uint32_t smem_dst, uint32_t cols) {
  asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_dst), "r"(cols) : "memory");
  asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
}
__device__ __forceinline__ void tmem_dealloc(uint32_t taddr, uint32_t cols) {
  asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(taddr), "r"(cols) : "memory");
}
// D[tmem] (+)= A[smem desc] * B[smem desc]; one thread issues it for the CTA
__device__ __forceinline__ void umma_f16(uint32_t tmem_d, uint64_t desc_a, uint64_t desc_b, uint32_t idesc, uint32_t accumulate) {
  asm volatile(
      "{\n\t.reg .pred p;\n\tsetp.ne.b32 p, %4, 0;\n\t"
      "tcgen05.mma.cta_group::1.kind::f16 [%0], %1, %2, %3, p;\n\t}" ::"r"(tmem_d),
      "l"(desc_a), "l"(desc_b), "r"(idesc), "r"(accumulate)
      : "memory");
}
// the mbarrier receives one arrival once every tensor-core instruction issued so far has completed
__device__ __forceinline__ void umma_commit(uint32_t bar) {
  asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(bar) : "memory");
}
__device__ __forceinline__ void tc_fence_after() { asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void tc_fence_before() { asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory"); }
// 32 consecutive accumulator columns of this thread's lane
__device__ __forceinline__ void tmem_ld32(uint32_t taddr, uint32_t (&r)[32]) {
  asm volatile(
      "tcgen05.ld.sync.aligned.32x32b.x32.b32 {%0,%1,%2,%3,%4,%5,%6,%7,%8,%9,%10,%11,%12,%13,%14,%15,%16,%17,%18,%19,%20,%21,%22,"
      "%23,%24,%25,%26,%27,%28,%29,%30,%31}, [%32];"
      : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7]), "=r"(r[8]), "=r"(r[9]),
        "=r"(r[10]), "=r"(r[11]), "=r"(r[12]), "=r"(r[13]), "=r"(r[14]), "=r"(r[15]), "=r"(r[16]), "=r"(r[17]), "=r"(r[18]),
        "=r"(r[19]), "=r"(r[20]), "=r"(r[21]), "=r"(r[22]), "=r"(r[23]), "=r"(r[24]), "=r"(r[25]), "=r"(r[26]), "=r"(r[27]),
        "=r"(r[28]), "=r"(r[29]), "=r"(r[30]), "=r"(r[31])
      : "r"(taddr)
      : "memory");
  asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory");
}

// Shared-memory matrix descriptor of a K-major tile whose rows are 128 bytes, 128-byte swizzled (what the
// tensor-map copy writes): 8-row groups 1024 bytes apart; descriptor version 1; swizzle mode 2.
__device__ __forceinline__ uint64_t smem_desc_k128(uint32_t smem_addr) {
  return (uint64_t)((smem_addr & 0x3FFFFu) >> 4) | ((uint64_t)1 << 16) | ((uint64_t)(1024 >> 4) << 32) | ((uint64_t)1 << 46) |
         ((uint64_t)2 << 61);
}
// Instruction descriptor: fp32 accumulate, A and B of the 16-bit type (both K-major), N = 128, M = 128.
template <int DT, int N>
__device__ __forceinline__ uint32_t umma_idesc() {
  const uint32_t fmt = DT == MC_F16 ? 0u : 1u;
  return (1u << 4) | (fmt << 7) | (fmt << 10) | ((uint32_t)(N >> 3) << 17) | ((uint32_t)(kPfTileM >> 4) << 24);
}

// NH = heads per CTA.  NH = 2: the tile is 128 tokens x 256 channels (one N = 256 instruction per K step, 256
// columns of tensor memory), the X tile feeds two heads -- a quarter less operand traffic through L2 per output
// element, which is what bounds the launch; the stages are 48 KB then, and the epilogue's row staging takes the
// stage memory over once the main loop is done (layer l-1's rows are fetched only then, head by head).
template <int DT, int NH>
__global__ void __launch_bounds__(kPfThreads, 2)
prefill_merge_kernel(const __grid_constant__ PrefillParams p, const __grid_constant__ CUtensorMap map_x,
                     const __grid_constant__ CUtensorMap map_wk, const __grid_constant__ CUtensorMap map_wv) {
  grid_dep_wait();
  grid_dep_launch();
  extern __shared__ unsigned char smem_raw[];
  unsigned char* smem = reinterpret_cast<unsigned char*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
  constexpr int STAGE_BYTES = (kPfTileM + NH * kPfTileN) * kPfTileK * 2;
  constexpr int TMEM_COLS = NH * kPfTmemCols;
  uint64_t* bars = reinterpret_cast<uint64_t*>(smem + kPfStages * STAGE_BYTES);  // full[stages], empty[stages], accum
  uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(bars + 2 * kPfStages + 1);
  volatile int* s_abort = reinterpret_cast<volatile int*>(tmem_slot + 1);
  // [4 warps][32 rows][kPfEpiRow]: row staging of the epilogue (NH = 2: over the stages, after the main loop)
  unsigned char* epi = NH == 1 ? smem + kPfStages * STAGE_BYTES + 256 : smem;
  const uint32_t stage0 = smem_u32(smem);
  const uint32_t full0 = smem_u32(bars), empty0 = full0 + 8 * kPfStages, accum_bar = empty0 + 8 * kPfStages;
  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;

  const int H = p.g.n_kv_heads;
  // Tile order: the CTAs that run at the same time should share operands in L2.  CTAs are numbered in
  // groups of mt_group token tiles x ht_group (tensor, head) columns -- inside a group the token tile runs
  // fastest, the groups of one band of token tiles follow each other -- so a group touches mt_group X
  // tiles and ht_group W slices (a few tens of MB), each used by many of its CTAs, and the X tiles of a
  // band stay resident while the W slices cycle.
  const int per_group = p.mt_group * p.ht_group;
  const int grp = blockIdx.x / per_group, within = blockIdx.x % per_group;
  const int mt = (grp / p.n_htg) * p.mt_group + within % p.mt_group;
  const int ht = (grp % p.n_htg) * p.ht_group + within / p.mt_group;
  if (mt >= p.n_mtiles) return;
  const int tensor = ht / p.n_hgroups, head0 = (ht % p.n_hgroups) * NH;
  const int tiles_per_seq = p.x_seq_stride / kPfTileM;
  const int b = mt / tiles_per_seq, tile = mt % tiles_per_seq;
  const int tok0 = tile * kPfTileM;
  const int n = checked_len(p.g, b, p.status);
  if (tok0 >= n) return;  // (the whole CTA: nothing has been set up yet)

  if (tid == 0) {
    for (int s = 0; s < kPfStages; ++s) {
      mbar_init(full0 + 8 * s, 1);
      mbar_init(empty0 + 8 * s, 1);
    }
    mbar_init(accum_bar, 1);
    *s_abort = 0;
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  if (warp == 1) tmem_alloc(smem_u32(tmem_slot), TMEM_COLS);
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem_d = *tmem_slot;
  const int n_kb = p.d_model / kPfTileK;

  if (warp == 0) {
    // ===================== producer: tensor-map copies of the X and W tiles =====================
    if (lane == 0) {
      const CUtensorMap* map_w = tensor ? &map_wv : &map_wk;
      for (int kb = 0; kb < n_kb; ++kb) {
        const int s = kb % kPfStages;
        if (kb >= kPfStages && !mbar_wait(empty0 + 8 * s, ((kb / kPfStages) - 1) & 1, s_abort, p.status)) break;
        const uint32_t bar = full0 + 8 * s;
        mbar_expect_tx(bar, (uint32_t)STAGE_BYTES);
        tma_load_2d(stage0 + s * STAGE_BYTES, &map_x, kb * kPfTileK, b * p.x_seq_stride + tok0, bar);
        tma_load_2d(stage0 + s * STAGE_BYTES + kPfTileM * kPfTileK * 2, map_w, kb * kPfTileK, head0 * kPfTileN, bar);
      }
    }
  } else if (warp == 1) {
    // ===================== tensor-core issue =====================
    if (lane == 0) {
      const uint32_t idesc = umma_idesc<DT, NH * kPfTileN>();
      bool ok = true;
      for (int kb = 0; kb < n_kb && ok; ++kb) {
        const int s = kb % kPfStages;
        if (!mbar_wait(full0 + 8 * s, (kb / kPfStages) & 1, s_abort, p.status)) { ok = false; break; }
        tc_fence_after();
        const uint64_t da = smem_desc_k128(stage0 + s * STAGE_BYTES);
        const uint64_t db = smem_desc_k128(stage0 + s * STAGE_BYTES + kPfTileM * kPfTileK * 2);
#pragma unroll
        for (int k = 0; k < kPfTileK / 16; ++k)  // 16 elements (32 bytes) per instruction along K
          umma_f16(tmem_d, da + (uint64_t)(2 * k), db + (uint64_t)(2 * k), idesc, (kb > 0 || k > 0) ? 1u : 0u);
        umma_commit(empty0 + 8 * s);  // the stage is free once these have read it
      }
      umma_commit(accum_bar);  // (also on the abort path: the epilogue's wait then ends early)
    }
  } else {
    // ===================== epilogue: one token row per thread =====================
    // Global memory is touched a row at a time by sixteen lanes (whole 256-byte rows), the arithmetic
    // wants a row per thread: the rows pass through a padded staging area in shared memory.
    const int q = warp & 3;            // the quarter of the tensor memory's lanes this warp may read
    const int m = q * 32 + lane;       // row of the tile
    const int tok = tok0 + m;
    const int ps = p.g.page_size, shift = p.g.page_shift;
    int page = -1;
    if (tok < n) page = checked_page(p.g, b, tok >> shift, p.status);
    const int tk = tok & (ps - 1);
    unsigned char* my = epi + q * kPfEpiWarp;  // (head hh of the CTA: + hh * 4 * kPfEpiWarp)
    const int r_half = lane >> 4, ch16 = lane & 15;
    // layer l-1's rows of head `hd` into its staging area, sixteen lanes per row
    auto fetch_a = [&](int hd) {
      unsigned char* my = epi + (hd - head0) * 4 * kPfEpiWarp + q * kPfEpiWarp;
      const int prow_h = page >= 0 ? (page * H + hd) * ps + tk : -1;
#pragma unroll 4
      for (int i = 0; i < 16; ++i) {
        const int r = 2 * i + r_half;
        const int pr = __shfl_sync(0xffffffffu, prow_h, r);
        if (pr >= 0)
          *reinterpret_cast<uint4*>(my + r * kPfEpiRow + ch16 * 16) =
              ld_stream16(p.a_pool[tensor] + (size_t)pr * kRowBytes + ch16 * 16);
      }
      __syncwarp();
    };
    if (NH == 1) fetch_a(head0);  // ... while the tensor cores are still busy (its own staging area)
    const bool ok_wait = mbar_wait(accum_bar, 0, s_abort, p.status);
    tc_fence_after();
    if (NH > 1) {  // (the stages are free: every tensor-core instruction has completed; both heads' rows are
      fetch_a(head0);  //  requested now, the second head's arrive under the first head's passes)
      fetch_a(head0 + 1);
    }
#pragma unroll 1
    for (int hh = 0; hh < NH; ++hh) {
    const int head = head0 + hh;
    const int prow = page >= 0 ? (page * H + head) * ps + tk : -1;  // row index inside a layer pool (-1: no such row)
    my = epi + hh * 4 * kPfEpiWarp + q * kPfEpiWarp;
    const bool live = ok_wait && !*s_abort && prow >= 0;
    // Layer l's row = the accumulators rounded once to the storage type (what the model would have cached).
    // Neither row is held in registers across the three passes of the merge (two 64-register copies would not
    // leave room for two CTAs per SM): layer l's 32-channel blocks are read from tensor memory again in every
    // pass -- the rounding is deterministic, so every pass sees the same bits --, layer l-1's row is read from
    // the staging area, which the last pass overwrites, chunk by chunk, with the merged row.
    // (tcgen05.ld is warp-wide: every lane runs the passes; only the stores depend on the lane having a row.)
    const unsigned char* my_row = my + lane * kPfEpiRow;
    auto load_c = [&](int j, uint32_t (&cj)[16]) {
      uint32_t r[32];
      tmem_ld32(tmem_d + ((uint32_t)(q * 32) << 16) + (uint32_t)(hh * kPfTmemCols + j * 32), r);
#pragma unroll
      for (int i = 0; i < 16; ++i) cj[i] = Elem<DT>::pack(__uint_as_float(r[2 * i]), __uint_as_float(r[2 * i + 1]));
    };
    float dmin = __int_as_float(0x7f800000), dmax = 0.f;
    {
      float aa = 0.f, cc = 0.f;
#pragma unroll 1
      for (int j = 0; j < 4; ++j) {
        uint32_t cj[16];
        load_c(j, cj);
#pragma unroll
        for (int cq = 0; cq < 4; ++cq) {
          const uint4 av = *reinterpret_cast<const uint4*>(my_row + (4 * j + cq) * 16);
          const uint32_t aw4[4] = {av.x, av.y, av.z, av.w};
#pragma unroll
          for (int i = 0; i < 4; ++i) {
            const float2 a = Elem<DT>::unpack(aw4[i]), c = Elem<DT>::unpack(cj[4 * cq + i]);
            aa = fmaf(a.x, a.x, fmaf(a.y, a.y, aa));
            cc = fmaf(c.x, c.x, fmaf(c.y, c.y, cc));
          }
        }
      }
      const float ia = aa > 0.f ? rsqrtf(aa) : 0.f, ic = cc > 0.f ? rsqrtf(cc) : 0.f;
      // |u - v|^2 and |u + v|^2 channel by channel (no cancellation at either end)
      float sm = 0.f, sp = 0.f;
#pragma unroll 1
      for (int j = 0; j < 4; ++j) {
        uint32_t cj[16];
        load_c(j, cj);
#pragma unroll
        for (int cq = 0; cq < 4; ++cq) {
          const uint4 av = *reinterpret_cast<const uint4*>(my_row + (4 * j + cq) * 16);
          const uint32_t aw4[4] = {av.x, av.y, av.z, av.w};
#pragma unroll
          for (int i = 0; i < 4; ++i) {
            const float2 a = Elem<DT>::unpack(aw4[i]), c = Elem<DT>::unpack(cj[4 * cq + i]);
            const float ux = a.x * ia, uy = a.y * ia;
            const float mx = fmaf(-c.x, ic, ux), my_ = fmaf(-c.y, ic, uy), px = fmaf(c.x, ic, ux), py = fmaf(c.y, ic, uy);
            sm = fmaf(mx, mx, fmaf(my_, my_, sm));
            sp = fmaf(px, px, fmaf(py, py, sp));
          }
        }
      }
      float ta = p.ta, tc = p.tc;
      row_t(p.t_mode, aa, cc, ta, tc);
      const RowScalars s = slerp_scalars(aa, cc, sm, sp, ta, tc);
      // a token that may end up unmerged (Eq. 4) keeps its raw row of layer l
      const bool keep_raw = live && s.d > p.d_hint;
      uint4* cp = reinterpret_cast<uint4*>(p.c_pool[tensor] + (size_t)max(prow, 0) * kRowBytes);
      float ee = 0.f;
#pragma unroll 1
      for (int j = 0; j < 4; ++j) {
        uint32_t cj[16];
        load_c(j, cj);
#pragma unroll
        for (int cq = 0; cq < 4; ++cq) {  // 16-byte chunk 4 j + cq of the row = channels [8 (4 j + cq), + 8)
          const int ch = 4 * j + cq;
          const uint4 av = *reinterpret_cast<const uint4*>(my_row + ch * 16);
          const uint32_t aw4[4] = {av.x, av.y, av.z, av.w};
          uint32_t w[4];
#pragma unroll
          for (int i = 0; i < 4; ++i) {
            const float2 a = Elem<DT>::unpack(aw4[i]), c = Elem<DT>::unpack(cj[4 * cq + i]);
            w[i] = Elem<DT>::pack(fmaf(s.fa, a.x, s.fc * c.x), fmaf(s.fa, a.y, s.fc * c.y));
            const float2 r = Elem<DT>::unpack(w[i]);  // the stored value: Eq. 2 divides by its length
            ee = fmaf(r.x, r.x, fmaf(r.y, r.y, ee));
          }
          *reinterpret_cast<uint4*>(my + lane * kPfEpiRow + ch * 16) = make_uint4(w[0], w[1], w[2], w[3]);
          if (keep_raw) cp[ch] = make_uint4(cj[4 * cq], cj[4 * cq + 1], cj[4 * cq + 2], cj[4 * cq + 3]);
        }
      }
      if (live) {
        const float il = ee > 0.f ? 1.0f / sqrtf(ee) : 0.f;
        char* tile_p = p.e_pool[tensor] + ((size_t)page * H + head) * tile_bytes(ps);
        float* scp = reinterpret_cast<float*>(tile_p + ps * kRowBytes) + tk;
        scp[0] = s.na * il;
        scp[ps] = s.nc * il;
        p.dist[(((size_t)page * H + head) * 2 + tensor) * ps + tk] = s.d;
        dmin = dmax = s.d;
      }
    }
    __syncwarp();
    // the merged rows leave: sixteen lanes per row
    const int page_live = live ? page : -1;
#pragma unroll 4
    for (int i = 0; i < 16; ++i) {
      const int r = 2 * i + r_half;
      const int pg = __shfl_sync(0xffffffffu, page_live, r);
      if (pg >= 0) {
        const int tk_r = (tok0 + q * 32 + r) & (ps - 1);
        // (chunk ch16 goes to its place in the tile's chunk order: the sixteen lanes still cover the whole row)
        st_stream16(p.e_pool[tensor] + ((size_t)pg * H + head) * tile_bytes(ps) + tk_r * kRowBytes + chunk_pos(tk_r, ch16) * 16,
                    *reinterpret_cast<const uint4*>(my + r * kPfEpiRow + ch16 * 16));
      }
    }
#pragma unroll
    for (int o = 16; o; o >>= 1) {
      dmin = fminf(dmin, __shfl_xor_sync(0xffffffffu, dmin, o));
      dmax = fmaxf(dmax, __shfl_xor_sync(0xffffffffu, dmax, o));
    }
    if (lane == 0 && dmin != __int_as_float(0x7f800000)) {
      const int seg = (tensor * p.g.batch + b) * H + head;
      atomicMin(&p.seg_minmax[2 * seg], __float_as_uint(dmin));
      atomicMax(&p.seg_minmax[2 * seg + 1], __float_as_uint(dmax));
    }
    __syncwarp();  // (the staging area is reused by the next head)
    }
  }
  // ---- every path ends here: the accumulators are no longer needed, the tensor memory goes back
  tc_fence_before();
  __syncthreads();
  if (warp == 1) {
    tc_fence_after();
    tmem_dealloc(tmem_d, TMEM_COLS);
  }
  if (*s_abort) {
    for (int x = 0; x < 2000; ++x) __nanosleep(1000);  // let copies in flight land before the CTA's memory is released
  }
}

// ---- host side ----------------------------------------------------------------------------------
typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*, const cuuint64_t*,
                                  const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave, CUtensorMapSwizzle,
                                  CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

static EncodeTiledFn encode_tiled_fn() {
  static std::mutex mu;
  static EncodeTiledFn fn = nullptr;
  std::lock_guard<std::mutex> lock(mu);
  if (fn == nullptr) {
    void* ptr = nullptr;
    cudaDriverEntryPointQueryResult qres;
    if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &ptr, cudaEnableDefault, &qres) == cudaSuccess &&
        qres == cudaDriverEntryPointSuccess)
      fn = reinterpret_cast<EncodeTiledFn>(ptr);
  }
  return fn;
}

// A [rows][cols] 16-bit row-major matrix, copied in boxes of box_rows rows x 64 columns with the 128-byte swizzle.
static mc_status make_map(CUtensorMap* map, int dtype, const void* base, uint64_t rows, uint64_t cols, int box_rows) {
  EncodeTiledFn fn = encode_tiled_fn();
  if (fn == nullptr) return MC_ERR_UNSUPPORTED;
  const cuuint64_t dims[2] = {cols, rows};
  const cuuint64_t strides[1] = {cols * 2};
  const cuuint32_t box[2] = {(cuuint32_t)kPfTileK, (cuuint32_t)box_rows};
  const cuuint32_t estr[2] = {1, 1};
  const CUresult r = fn(map, dtype == MC_F16 ? CU_TENSOR_MAP_DATA_TYPE_FLOAT16 : CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2,
                        const_cast<void*>(base), dims, strides, box, estr, CU_TENSOR_MAP_INTERLEAVE_NONE,
                        CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_128B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
  if (r != CUDA_SUCCESS) {
    set_cuda_error(cudaErrorInvalidValue, "cuTensorMapEncodeTiled");
    return MC_ERR_CUDA;
  }
  return MC_OK;
}

mc_status launch_prefill_merge(const mc_config* cfg, const mc_batch* bt, const Geom& g, const mc_projection* proj,
                               const mc_layer_kv* lm1, const mc_layer_kv* l, const mc_pair_cache* out, float d_hint,
                               cudaStream_t stream) {
  if (bt->batch == 0) return MC_OK;
  CUtensorMap map_x, map_wk, map_wv;
  const uint64_t x_rows = (uint64_t)bt->batch * proj->x_seq_stride;
  const uint64_t w_rows = (uint64_t)cfg->n_kv_heads * kPfTileN;
  const int nh = cfg->n_kv_heads % 2 == 0 ? 2 : 1;  // heads per CTA
  if (mc_status st = make_map(&map_x, cfg->dtype, proj->x, x_rows, proj->d_model, kPfTileM)) return st;
  if (mc_status st = make_map(&map_wk, cfg->dtype, proj->w_k, w_rows, proj->d_model, nh * kPfTileN)) return st;
  if (mc_status st = make_map(&map_wv, cfg->dtype, proj->w_v, w_rows, proj->d_model, nh * kPfTileN)) return st;
  PrefillParams pp;
  pp.g = g;
  pp.a_pool[0] = (const char*)lm1->k_pool;
  pp.a_pool[1] = (const char*)lm1->v_pool;
  pp.c_pool[0] = (char*)l->k_pool;
  pp.c_pool[1] = (char*)l->v_pool;
  pp.e_pool[0] = (char*)out->e_k;
  pp.e_pool[1] = (char*)out->e_v;
  pp.dist = out->dist;
  pp.seg_minmax = reinterpret_cast<unsigned*>(out->seg_minmax);
  pp.status = out->status;
  pp.x_seq_stride = proj->x_seq_stride;
  pp.d_model = proj->d_model;
  pp.ta = (float)(1.0 - cfg->t);
  pp.tc = (float)cfg->t;
  pp.t_mode = cfg->t_mode;
  pp.d_hint = d_hint;
  // stages, barriers, row staging (two heads per CTA: the staging lives in the stages)
  const size_t smem = nh == 1 ? 1024 + (size_t)kPfStages * kPfStageBytes + 256 + 4 * (size_t)kPfEpiWarp
                              : 1024 + (size_t)kPfStages * (kPfTileM + 2 * kPfTileN) * kPfTileK * 2 + 256;
  pp.n_mtiles = bt->batch * (proj->x_seq_stride / kPfTileM);
  pp.n_hgroups = cfg->n_kv_heads / nh;
  const int n_ht = 2 * pp.n_hgroups;
  pp.ht_group = 1;
  for (int dv = 1; dv <= 16; ++dv)
    if (n_ht % dv == 0) pp.ht_group = dv;  // the largest divisor of the column count up to 16
  pp.n_htg = n_ht / pp.ht_group;
  pp.mt_group = std::min(32, pp.n_mtiles);
  const long long n_ctas = (long long)((pp.n_mtiles + pp.mt_group - 1) / pp.mt_group) * pp.n_htg * pp.mt_group * pp.ht_group;
  if (n_ctas > 0x7fffffffLL) return MC_ERR_SHAPE;
  const dim3 grid((unsigned)n_ctas);
  void (*kern)(const PrefillParams, const CUtensorMap, const CUtensorMap, const CUtensorMap) =
      cfg->dtype == MC_F16 ? (nh == 2 ? prefill_merge_kernel<MC_F16, 2> : prefill_merge_kernel<MC_F16, 1>)
                           : (nh == 2 ? prefill_merge_kernel<MC_BF16, 2> : prefill_merge_kernel<MC_BF16, 1>);
  MC_CUDA_CHECK(cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem));
  MC_CUDA_CHECK(launch_pdl(kern, grid, dim3(kPfThreads), smem, stream, pp, map_x, map_wk, map_wv));
  MC_CUDA_CHECK(cudaGetLastError());
  return MC_OK;
}

}  // namespace mc
