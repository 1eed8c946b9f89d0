// Single-query decode attention straight over the compressed pair cache
// (Algorithm 2 "MiniCache Decoding": rescale by the layer's magnitude, put the retained rows
// back, append the new token, softmax(q K^T) V), with the restore folded into the kernel:
//
//   q . (g_i e_i) = g_i (q . e_i)            the K magnitude scales the score
//   sum_i p_i (g_i e_i) = sum_i (p_i g_i) e_i  the V magnitude scales the probability
//
// so the shared direction rows are streamed once, untouched, and a retained token only
// replaces one score (K) or one term of the sum (V).
//
// Work item = (sequence, kv head, split of the token axis).  One producer thread streams the
// page tiles of the split with TMA (128-byte swizzled boxes, mbarrier pipeline): first all K
// tiles, then all V tiles.  Four consumer warps run both contractions on the tensor cores with
// the query rows of the kv head's group (and, in pair mode, of both layers) as the padded M
// tile: scores -> shared memory -> split-local softmax -> P V.  Partial (m, l, o) per split are
// merged by attn_combine_kernel.
#include <cuda.h>

#include "mc_common.cuh"
#include "mc_kernels.h"

namespace mc {

constexpr int kTile = 64;  // tokens per pipeline stage
constexpr int kStages = 4;
constexpr int kConsumerWarps = 4;
constexpr int kConsumerThreads = kConsumerWarps * 32;
constexpr int kAttnThreads = kConsumerThreads + 64;  // + producer warp + lookup warp
constexpr int kMaxRows = 8;                          // query rows per work item (M tile rows used)
constexpr int kTileBytes = kTile * kRowBytes;        // 16 KB
constexpr int kStageScaleBytes = 1024;
constexpr int kStageBytes = kTileBytes + kStageScaleBytes;
constexpr int kMaxSplit = 1024;
constexpr uint32_t kWaitLimit = 1u << 22;

struct AttnParams {
  Geom g;
  const float* scale;
  const int32_t* ret_count;
  const int32_t* ret_offset;
  const int32_t* ret_index;
  const char* ret_rows;
  const char* q;
  const char* k_new;
  const char* v_new;
  float* part_o;   // [n_sets][batch][Hq][n_splits][128]
  float* part_ml;  // [n_sets][batch][Hq][n_splits][2]
  int32_t* status;
  float scale_log2;  // sm_scale * log2(e)
  int layer_sel;
  int n_sets;
  int nq;    // query heads per kv head
  int rows;  // n_sets * nq
  int n_q_heads;
  int split_len;
  int n_splits;
};

// ---- PTX wrappers -----------------------------------------------------------------------------
__device__ __forceinline__ uint32_t smem_u32(const void* p) { return (uint32_t)__cvta_generic_to_shared(p); }
__device__ __forceinline__ void mbar_init(uint32_t bar, int count) {
  asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(bar), "r"(count) : "memory");
}
__device__ __forceinline__ void mbar_expect_tx(uint32_t bar, uint32_t bytes) {
  asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(bar), "r"(bytes) : "memory");
}
__device__ __forceinline__ void mbar_arrive(uint32_t bar) {
  asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(bar) : "memory");
}
__device__ __forceinline__ bool mbar_try_wait(uint32_t bar, uint32_t parity) {
  uint32_t ok;
  asm volatile(
      "{\n\t.reg .pred p;\n\tmbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\tselp.u32 %0, 1, 0, p;\n\t}"
      : "=r"(ok)
      : "r"(bar), "r"(parity)
      : "memory");
  return ok != 0;
}
__device__ __forceinline__ void tma_load_2d(uint32_t dst, const CUtensorMap* tm, int x, int y, uint32_t bar) {
  asm volatile(
      "cp.async.bulk.tensor.2d.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%2, %3}], [%4];" ::"r"(
          dst),
      "l"(tm), "r"(x), "r"(y), "r"(bar)
      : "memory");
}
__device__ __forceinline__ void bulk_load(uint32_t dst, const void* src, uint32_t bytes, uint32_t bar) {
  asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];" ::"r"(dst),
               "l"(src), "r"(bytes), "r"(bar)
               : "memory");
}
__device__ __forceinline__ void ldsm_x4(uint32_t addr, uint32_t& r0, uint32_t& r1, uint32_t& r2, uint32_t& r3) {
  asm volatile("ldmatrix.sync.aligned.m8n8.x4.shared.b16 {%0,%1,%2,%3}, [%4];"
               : "=r"(r0), "=r"(r1), "=r"(r2), "=r"(r3)
               : "r"(addr));
}
__device__ __forceinline__ void ldsm_x4_t(uint32_t addr, uint32_t& r0, uint32_t& r1, uint32_t& r2, uint32_t& r3) {
  asm volatile("ldmatrix.sync.aligned.m8n8.x4.trans.shared.b16 {%0,%1,%2,%3}, [%4];"
               : "=r"(r0), "=r"(r1), "=r"(r2), "=r"(r3)
               : "r"(addr));
}
// D += A(16x16, rows 8..15 zero) * B(16x8); only the two accumulator registers of rows 0..7 matter
// to the caller but the instruction carries all four.
template <int DT>
__device__ __forceinline__ void mma_16816(float (&c)[4], uint32_t a0, uint32_t a2, uint32_t b0, uint32_t b1) {
  const uint32_t z = 0u;
  if (DT == MC_F16) {
    asm volatile(
        "mma.sync.aligned.m16n8k16.row.col.f32.f16.f16.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%0,%1,%2,%3};"
        : "+f"(c[0]), "+f"(c[1]), "+f"(c[2]), "+f"(c[3])
        : "r"(a0), "r"(z), "r"(a2), "r"(z), "r"(b0), "r"(b1));
  } else {
    asm volatile(
        "mma.sync.aligned.m16n8k16.row.col.f32.bf16.bf16.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%0,%1,%2,%3};"
        : "+f"(c[0]), "+f"(c[1]), "+f"(c[2]), "+f"(c[3])
        : "r"(a0), "r"(z), "r"(a2), "r"(z), "r"(b0), "r"(b1));
  }
}
__device__ __forceinline__ void consumer_sync() { asm volatile("bar.sync 1, %0;" ::"n"(kConsumerThreads) : "memory"); }

// Bounded wait: gives up after kWaitLimit polls, records it, and makes every later wait of the
// CTA (and of CTAs that start afterwards) return at once.
__device__ __forceinline__ bool mbar_wait(uint32_t bar, uint32_t parity, volatile int* s_abort, int32_t* status) {
  if (*s_abort) return false;
  for (uint32_t it = 0; it < kWaitLimit; ++it) {
    if (mbar_try_wait(bar, parity)) return true;
    if (it > 64) __nanosleep(40);
    if ((it & 1023) == 1023 && (*s_abort || (*(volatile int32_t*)status & MC_FLAG_WAIT_TIMEOUT))) break;
  }
  *s_abort = 1;
  atomicOr(status, MC_FLAG_WAIT_TIMEOUT);
  return false;
}

// Address of 16-byte chunk `chunk` (0..15 over the 128 channels) of tile row `tk` inside a stage.
// A stage holds, per page j and channel half, one TMA box [page_size rows][128 bytes] written
// with the 128-byte swizzle: chunk c of row r sits at chunk position c ^ (r & 7).
__device__ __forceinline__ uint32_t tile_addr(uint32_t stage, int tk, int chunk, int page_shift) {
  const int j = tk >> page_shift;
  const int r = tk & ((1 << page_shift) - 1);
  const int half = chunk >> 3;
  return stage + (uint32_t)(((j * 2 + half) << page_shift) * 128 + r * 128 + (((chunk & 7) ^ (r & 7)) << 4));
}

template <int DT>
__global__ void __launch_bounds__(kAttnThreads) attn_split_kernel(const __grid_constant__ CUtensorMap tm_k,
                                                                 const __grid_constant__ CUtensorMap tm_v,
                                                                 const AttnParams p) {
  const int split = blockIdx.x, g = blockIdx.y, b = blockIdx.z;
  const int n = p.g.seq_lens[b];
  const int n_splits_b = max(1, (n + p.split_len - 1) / p.split_len);
  if (split >= n_splits_b) return;
  const int split_start = split * p.split_len;
  const int n_tok = max(0, min(n, split_start + p.split_len) - split_start);  // cached tokens of this split
  const bool has_new = (p.k_new != nullptr) && (split == n_splits_b - 1);
  const int n_cols = n_tok + (has_new ? 1 : 0);
  const int T = (n_tok + kTile - 1) / kTile;
  const int ps = p.g.page_size, shift = p.g.page_shift;
  const int H = p.g.n_kv_heads;
  const int nslots = p.n_sets;
  const int rows = p.rows;
  const int s_stride = p.split_len + 8;

  extern __shared__ unsigned char smem_raw[];
  unsigned char* smem = reinterpret_cast<unsigned char*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
  unsigned char* stages = smem;
  float* S = reinterpret_cast<float*>(smem + kStages * kStageBytes);       // [kMaxRows][s_stride]
  float* O_s = S + kMaxRows * s_stride;                                    // [kMaxRows][128]
  uint32_t* q_s = reinterpret_cast<uint32_t*>(O_s + kMaxRows * kHeadDim);  // [kMaxRows][64] packed pairs
  int* pages_s = reinterpret_cast<int*>(q_s + kMaxRows * 64);              // [kMaxSplit / 16]
  float* m_s = reinterpret_cast<float*>(pages_s + kMaxSplit / 16);         // [kMaxRows]
  float* l_s = m_s + kMaxRows;
  int* look_s = reinterpret_cast<int*>(l_s + kMaxRows);  // k_lo, k_hi, v_lo, v_hi
  volatile int* s_abort = look_s + 4;
  uint64_t* bars = reinterpret_cast<uint64_t*>(look_s + 8);  // full[kStages], empty[kStages], lookup
  const uint32_t full0 = smem_u32(bars), empty0 = full0 + 8 * kStages, lookbar = full0 + 16 * kStages;
  const uint32_t stage0 = smem_u32(stages);

  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;

  // ---- prologue: barriers, page ids, query rows -------------------------------------------------
  if (tid == 0) {
    for (int s = 0; s < kStages; ++s) {
      mbar_init(full0 + 8 * s, 1);
      mbar_init(empty0 + 8 * s, kConsumerWarps);
    }
    mbar_init(lookbar, 1);
    *s_abort = 0;
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  {
    const int first_slot = split_start >> shift;
    const int n_pg = (n_tok + ps - 1) >> shift;
    for (int i = tid; i < n_pg; i += kAttnThreads)
      pages_s[i] = p.g.block_table[(size_t)b * p.g.max_pages_per_seq + first_slot + i];
    // query rows: row r = set * nq + rq  ->  q[set][b][g * nq + rq][:]
    for (int i = tid; i < kMaxRows * 64; i += kAttnThreads) {
      const int r = i >> 6, w = i & 63;
      uint32_t v = 0;
      if (r < rows) {
        const int set = r / p.nq, rq = r - set * p.nq;
        const size_t qrow = ((size_t)set * p.g.batch + b) * p.n_q_heads + g * p.nq + rq;
        v = reinterpret_cast<const uint32_t*>(p.q)[qrow * 64 + w];
      }
      q_s[i] = v;
    }
  }
  __syncthreads();

  const int seg_k = b * H + g;
  const int seg_v = (p.g.batch + b) * H + g;

  if (warp == kConsumerWarps) {
    // ===================== producer =====================
    if (lane == 0) {
      const uint32_t page_bytes = (uint32_t)ps * kRowBytes + (uint32_t)nslots * ps * 4;
      for (int it = 0; it < 2 * T; ++it) {
        const int phase = it >= T ? 1 : 0;
        const int t = it - phase * T;
        const int s = it % kStages;
        if (it >= kStages && !mbar_wait(empty0 + 8 * s, ((it / kStages) - 1) & 1, s_abort, p.status)) break;
        const int tok0 = t * kTile;
        const int n_pg = min(kTile >> shift, (n_tok - tok0 + ps - 1) >> shift);
        const uint32_t bar = full0 + 8 * s;
        const uint32_t sbase = stage0 + s * kStageBytes;
        mbar_expect_tx(bar, n_pg * page_bytes);
        const CUtensorMap* tm = phase ? &tm_v : &tm_k;
        for (int j = 0; j < n_pg; ++j) {
          const int page = pages_s[(tok0 >> shift) + j];
          const int y = (page * H + g) * ps;
          tma_load_2d(sbase + (uint32_t)((j * 2) << shift) * 128, tm, 0, y, bar);
          tma_load_2d(sbase + (uint32_t)((j * 2 + 1) << shift) * 128, tm, 64, y, bar);
          const int slot = phase * 2 + (nslots == 2 ? 0 : p.layer_sel);
          const float* src = p.scale + (((size_t)page * H + g) * 4 + slot) * ps;
          bulk_load(sbase + kTileBytes + (uint32_t)j * nslots * ps * 4, src, (uint32_t)nslots * ps * 4, bar);
        }
      }
    }
    return;
  }
  if (warp == kConsumerWarps + 1) {
    // ===================== retained-list lookup =====================
    // lane 0: K segment, lane 1: V segment.  Range of list entries whose token lies in this split.
    if (lane < 2) {
      const int seg = lane == 0 ? seg_k : seg_v;
      const int cnt = p.ret_count[seg];
      const int off = p.ret_offset[seg];
      int lo = 0, hi = cnt;  // first entry with token >= split_start
      while (lo < hi) {
        const int mid = (lo + hi) >> 1;
        if (p.ret_index[off + mid] < split_start) lo = mid + 1; else hi = mid;
      }
      const int first = lo;
      hi = cnt;  // first entry with token >= split_start + n_tok
      while (lo < hi) {
        const int mid = (lo + hi) >> 1;
        if (p.ret_index[off + mid] < split_start + n_tok) lo = mid + 1; else hi = mid;
      }
      look_s[lane * 2] = off + first;
      look_s[lane * 2 + 1] = off + lo;
    }
    __syncwarp();
    if (lane == 0) mbar_arrive(lookbar);  // release: the writes above are visible to waiters
    return;
  }

  // ===================== consumers =====================
  const int row = lane >> 2;         // M-tile row of this thread's fragments
  const int colp = (lane & 3) * 2;   // column pair inside an 8-wide n tile
  const int slot_row = (nslots == 2 && row < rows) ? row / p.nq : 0;

  // ---- K phase: S[r][i] = log2e * sm_scale * g_i * (q_r . e_i) -----------------------------------
  {
    uint32_t qa0[8], qa2[8];
#pragma unroll
    for (int ks = 0; ks < 8; ++ks) {
      qa0[ks] = q_s[row * 64 + ks * 8 + (lane & 3)];
      qa2[ks] = q_s[row * 64 + ks * 8 + 4 + (lane & 3)];
    }
    const int tk_w = warp * 16;  // this warp's 16 tokens of every tile
    const int mi = lane >> 3, mr = lane & 7;
    for (int t = 0; t < T; ++t) {
      const int it = t, s = it % kStages;
      if (!mbar_wait(full0 + 8 * s, (it / kStages) & 1, s_abort, p.status)) break;
      const uint32_t sbase = stage0 + s * kStageBytes;
      const int valid = min(kTile, n_tok - t * kTile);
      if (tk_w < valid) {
        float acc0[4] = {0.f, 0.f, 0.f, 0.f}, acc1[4] = {0.f, 0.f, 0.f, 0.f};
        const int tk_m = tk_w + (mi >> 1) * 8 + mr;  // token row this lane addresses for ldmatrix
#pragma unroll
        for (int ks = 0; ks < 8; ++ks) {
          uint32_t r0, r1, r2, r3;
          ldsm_x4(tile_addr(sbase, tk_m, ks * 2 + (mi & 1), shift), r0, r1, r2, r3);
          mma_16816<DT>(acc0, qa0[ks], qa2[ks], r0, r1);
          mma_16816<DT>(acc1, qa0[ks], qa2[ks], r2, r3);
        }
        if (row < rows) {
          const float* sc = reinterpret_cast<const float*>(stages + s * kStageBytes + kTileBytes);
          const int j = tk_w >> shift, r = tk_w & (ps - 1);
          const float* scj = sc + (j * nslots + slot_row) * ps + r;
          float* srow = S + row * s_stride + t * kTile + tk_w;
          const float2 g0 = *reinterpret_cast<const float2*>(scj + colp);
          const float2 g1 = *reinterpret_cast<const float2*>(scj + 8 + colp);
          *reinterpret_cast<float2*>(srow + colp) =
              make_float2(acc0[0] * g0.x * p.scale_log2, acc0[1] * g0.y * p.scale_log2);
          *reinterpret_cast<float2*>(srow + 8 + colp) =
              make_float2(acc1[0] * g1.x * p.scale_log2, acc1[1] * g1.y * p.scale_log2);
        }
      }
      __syncwarp();
      if (lane == 0) mbar_arrive(empty0 + 8 * s);
    }
  }
  consumer_sync();

  // ---- retained K rows and the new token replace / add single scores ----------------------------
  const bool any_list = (p.ret_count[seg_k] | p.ret_count[seg_v]) != 0;
  int k_lo = 0, k_hi = 0, v_lo = 0, v_hi = 0;
  if (any_list) {
    mbar_wait(lookbar, 0, s_abort, p.status);
    k_lo = look_s[0];
    k_hi = look_s[1];
    v_lo = look_s[2];
    v_hi = look_s[3];
  }
  {
    const int n_extra = (k_hi - k_lo) + (has_new ? 1 : 0);
    for (int e = warp; e < n_extra; e += kConsumerWarps) {
      const bool is_new = e >= (k_hi - k_lo);
      const int col = is_new ? n_tok : p.ret_index[k_lo + e] - split_start;
      for (int r = 0; r < rows; ++r) {
        const int set = r / p.nq;
        const char* src;
        if (is_new)
          src = p.k_new + (((size_t)set * p.g.batch + b) * H + g) * kRowBytes;
        else
          src = p.ret_rows + ((size_t)(k_lo + e) * 2 + (nslots == 2 ? set : p.layer_sel)) * kRowBytes;
        const uint2 kv = *reinterpret_cast<const uint2*>(src + lane * 8);
        const uint2 qv = *reinterpret_cast<const uint2*>(q_s + r * 64 + lane * 2);
        const float2 k0 = Elem<DT>::unpack(kv.x), k1 = Elem<DT>::unpack(kv.y);
        const float2 q0 = Elem<DT>::unpack(qv.x), q1 = Elem<DT>::unpack(qv.y);
        float d = q0.x * k0.x + q0.y * k0.y + q1.x * k1.x + q1.y * k1.y;
        for (int o = 16; o; o >>= 1) d += __shfl_xor_sync(0xffffffffu, d, o);
        if (lane == 0) S[r * s_stride + col] = d * p.scale_log2;
      }
    }
  }
  consumer_sync();

  // ---- split-local softmax: S <- 2^(S - m), row sums --------------------------------------------
  for (int r = warp; r < rows; r += kConsumerWarps) {
    float* srow = S + r * s_stride;
    float m = -INFINITY;
    for (int c = lane; c < n_cols; c += 32) m = fmaxf(m, srow[c]);
    for (int o = 16; o; o >>= 1) m = fmaxf(m, __shfl_xor_sync(0xffffffffu, m, o));
    float l = 0.f;
    for (int c = lane; c < n_cols; c += 32) {
      const float e = exp2f(srow[c] - m);
      srow[c] = e;
      l += e;
    }
    for (int o = 16; o; o >>= 1) l += __shfl_xor_sync(0xffffffffu, l, o);
    if (lane == 0) {
      m_s[r] = m;
      l_s[r] = l;
    }
  }
  consumer_sync();

  // ---- retained V rows and the new token: their terms are added outside the tile loop ------------
  float o_ret[kMaxRows];
#pragma unroll
  for (int r = 0; r < kMaxRows; ++r) o_ret[r] = 0.f;
  {
    const int n_extra = (v_hi - v_lo) + (has_new ? 1 : 0);
    const unsigned short* rr = reinterpret_cast<const unsigned short*>(p.ret_rows);
    for (int e = 0; e < n_extra; ++e) {
      const bool is_new = e >= (v_hi - v_lo);
      const int col = is_new ? n_tok : p.ret_index[v_lo + e] - split_start;
      float val[2];
#pragma unroll
      for (int set = 0; set < 2; ++set) {
        unsigned short bits = 0;
        if (set < nslots) {
          if (is_new)
            bits = reinterpret_cast<const unsigned short*>(p.v_new)[(((size_t)set * p.g.batch + b) * H + g) * kHeadDim + tid];
          else
            bits = rr[((size_t)(v_lo + e) * 2 + (nslots == 2 ? set : p.layer_sel)) * kHeadDim + tid];
        }
        val[set] = Elem<DT>::unpack((uint32_t)bits).x;
      }
#pragma unroll
      for (int r = 0; r < kMaxRows; ++r)
        if (r < rows) o_ret[r] = fmaf(S[r * s_stride + col], val[nslots == 2 ? r / p.nq : 0], o_ret[r]);
    }
    if (v_hi > v_lo) {
      consumer_sync();
      for (int e = tid; e < (v_hi - v_lo); e += kConsumerThreads) {
        const int col = p.ret_index[v_lo + e] - split_start;
        for (int r = 0; r < rows; ++r) S[r * s_stride + col] = 0.f;
      }
      consumer_sync();
    }
  }

  // ---- V phase: O[r][:] = sum_i (P[r][i] g_i) e_i -----------------------------------------------
  float acc[4][4];
#pragma unroll
  for (int i = 0; i < 4; ++i)
#pragma unroll
    for (int k = 0; k < 4; ++k) acc[i][k] = 0.f;
  {
    const int mi = lane >> 3, mr = lane & 7;
    const int chunk0 = warp * 4;  // this warp owns channels [32 warp, 32 warp + 32)
    for (int t = 0; t < T; ++t) {
      const int it = T + t, s = it % kStages;
      if (!mbar_wait(full0 + 8 * s, (it / kStages) & 1, s_abort, p.status)) break;
      const uint32_t sbase = stage0 + s * kStageBytes;
      const int valid = min(kTile, n_tok - t * kTile);
      const int ksteps = (valid + 15) >> 4;
      // rows past the last cached token may hold anything (page tail, unloaded page): zero this
      // warp's channels there so that 0 * x stays 0 in the contraction
      for (int rz = valid + (lane >> 2); rz < ksteps * 16; rz += 8) {
        const uint32_t a = tile_addr(sbase, rz, chunk0 + (lane & 3), shift);
        asm volatile("st.shared.v4.u32 [%0], {%1,%1,%1,%1};" ::"r"(a), "r"(0u) : "memory");
      }
      __syncwarp();
      const float* sc = reinterpret_cast<const float*>(stages + s * kStageBytes + kTileBytes);
      for (int kk = 0; kk < ksteps; ++kk) {
        // A fragment: probabilities times the V magnitude, rounded to the storage type
        uint32_t a0 = 0u, a2 = 0u;
        if (row < rows) {
          const int tk = kk * 16;
          const int j = tk >> shift, r = tk & (ps - 1);
          const float* scj = sc + (j * nslots + slot_row) * ps + r;
          const float* srow = S + row * s_stride + t * kTile + tk;
          const float2 p0 = *reinterpret_cast<const float2*>(srow + colp);
          const float2 p1 = *reinterpret_cast<const float2*>(srow + 8 + colp);
          const float2 g0 = *reinterpret_cast<const float2*>(scj + colp);
          const float2 g1 = *reinterpret_cast<const float2*>(scj + 8 + colp);
          const int c0 = tk + colp;
          a0 = Elem<DT>::pack(c0 < valid ? p0.x * g0.x : 0.f, c0 + 1 < valid ? p0.y * g0.y : 0.f);
          a2 = Elem<DT>::pack(c0 + 8 < valid ? p1.x * g1.x : 0.f, c0 + 9 < valid ? p1.y * g1.y : 0.f);
        }
        const int tk_m = kk * 16 + (mi & 1) * 8 + mr;
#pragma unroll
        for (int np = 0; np < 2; ++np) {
          uint32_t r0, r1, r2, r3;
          ldsm_x4_t(tile_addr(sbase, tk_m, chunk0 + np * 2 + (mi >> 1), shift), r0, r1, r2, r3);
          mma_16816<DT>(acc[np * 2], a0, a2, r0, r1);
          mma_16816<DT>(acc[np * 2 + 1], a0, a2, r2, r3);
        }
      }
      asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
      __syncwarp();
      if (lane == 0) mbar_arrive(empty0 + 8 * s);
    }
  }
  if (row < rows) {
#pragma unroll
    for (int nt = 0; nt < 4; ++nt)
      *reinterpret_cast<float2*>(O_s + row * kHeadDim + warp * 32 + nt * 8 + colp) = make_float2(acc[nt][0], acc[nt][1]);
  }
  consumer_sync();

  // ---- partial results of this split --------------------------------------------------------------
#pragma unroll
  for (int r = 0; r < kMaxRows; ++r) {
    if (r < rows) {
      const int set = r / p.nq, rq = r - set * p.nq;
      const size_t prow = (((size_t)set * p.g.batch + b) * p.n_q_heads + g * p.nq + rq) * p.n_splits + split;
      p.part_o[prow * kHeadDim + tid] = O_s[r * kHeadDim + tid] + o_ret[r];
      if (tid == 0) {
        p.part_ml[prow * 2] = m_s[r];
        p.part_ml[prow * 2 + 1] = l_s[r];
      }
    }
  }
  if (*s_abort) {
    // give copies that may still be in flight time to land before the CTA's memory is released
    for (int i = 0; i < 2000; ++i) __nanosleep(1000);
  }
}

// Log-sum-exp merge of the split partials: out = sum_j 2^(m_j - M) o_j / sum_j 2^(m_j - M) l_j.
template <int DT>
__global__ void __launch_bounds__(128) attn_combine_kernel(const AttnParams p, unsigned short* out, float* lse) {
  const int hq = blockIdx.x, b = blockIdx.y, set = blockIdx.z;
  const int n = p.g.seq_lens[b];
  const int nsp = max(1, (n + p.split_len - 1) / p.split_len);
  const size_t prow0 = (((size_t)set * p.g.batch + b) * p.n_q_heads + hq) * p.n_splits;
  float M = -INFINITY;
  for (int j = 0; j < nsp; ++j) M = fmaxf(M, p.part_ml[(prow0 + j) * 2]);
  float L = 0.f, o = 0.f;
  for (int j = 0; j < nsp; ++j) {
    const float m = p.part_ml[(prow0 + j) * 2];
    const float w = m == -INFINITY ? 0.f : exp2f(m - M);
    L = fmaf(w, p.part_ml[(prow0 + j) * 2 + 1], L);
    o = fmaf(w, p.part_o[(prow0 + j) * kHeadDim + threadIdx.x], o);
  }
  const float res = L > 0.f ? o / L : 0.f;
  const size_t orow = ((size_t)set * p.g.batch + b) * p.n_q_heads + hq;
  const uint32_t packed = Elem<DT>::pack(res, 0.f);
  out[orow * kHeadDim + threadIdx.x] = (unsigned short)(packed & 0xffffu);
  if (lse != nullptr && threadIdx.x == 0)
    lse[orow] = L > 0.f ? (M + log2f(L)) * 0.69314718055994530942f : -INFINITY;
}

// ---- host side ------------------------------------------------------------------------------------
static int pick_split_len(const mc_config* cfg, const mc_batch* bt) {
  const long long items = (long long)bt->batch * cfg->n_kv_heads;
  int len = kMaxSplit;
  while (len > 128 && items * ((bt->max_seq_len + len - 1) / len) < 148 * 4) len >>= 1;
  return len;
}

static size_t attn_smem_bytes(int split_len) {
  return 1024 + (size_t)kStages * kStageBytes + (size_t)kMaxRows * (split_len + 8) * 4 + kMaxRows * kHeadDim * 4 +
         kMaxRows * 64 * 4 + (kMaxSplit / 16) * 4 + 2 * kMaxRows * 4 + 8 * 4 + (2 * kStages + 1) * 8 + 64;
}

size_t attn_workspace_bytes(const mc_config* cfg, const mc_batch* bt, int n_sets) {
  const int split_len = pick_split_len(cfg, bt);
  const size_t n_splits = (size_t)max(1, (bt->max_seq_len + split_len - 1) / split_len);
  const size_t prow = (size_t)n_sets * bt->batch * cfg->n_q_heads * n_splits;
  return align_up(prow * kHeadDim * 4, 256) + align_up(prow * 2 * 4, 256);
}

typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*,
                                  const cuuint64_t*, const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave,
                                  CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

static mc_status encode_pool_map(CUtensorMap* tm, const void* pool, int dtype, int64_t n_rows, int page_size) {
  static EncodeTiledFn fn = nullptr;
  if (fn == nullptr) {
    void* sym = nullptr;
    cudaDriverEntryPointQueryResult qr;
    MC_CUDA_CHECK(cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &sym, cudaEnableDefault, &qr));
    if (sym == nullptr || qr != cudaDriverEntryPointSuccess) {
      set_cuda_error(cudaErrorUnknown, "cuTensorMapEncodeTiled entry point not found");
      return MC_ERR_CUDA;
    }
    fn = reinterpret_cast<EncodeTiledFn>(sym);
  }
  const cuuint64_t dims[2] = {(cuuint64_t)kHeadDim, (cuuint64_t)n_rows};
  const cuuint64_t strides[1] = {(cuuint64_t)kRowBytes};
  const cuuint32_t box[2] = {64u, (cuuint32_t)page_size};
  const cuuint32_t estr[2] = {1u, 1u};
  const CUresult r = fn(tm, dtype == MC_F16 ? CU_TENSOR_MAP_DATA_TYPE_FLOAT16 : CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2,
                        const_cast<void*>(pool), dims, strides, box, estr, CU_TENSOR_MAP_INTERLEAVE_NONE,
                        CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                        CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
  if (r != CUDA_SUCCESS) {
    set_cuda_error(cudaErrorInvalidValue, "cuTensorMapEncodeTiled failed");
    return MC_ERR_CUDA;
  }
  return MC_OK;
}

mc_status launch_decode_attn(const mc_config* cfg, const mc_batch* bt, const Geom& g, const mc_pair_cache* pair,
                             int layer_sel, const void* q, const void* k_new, const void* v_new, float sm_scale,
                             void* out, float* lse, void* workspace, cudaStream_t stream) {
  if (bt->batch == 0) return MC_OK;
  AttnParams ap;
  ap.g = g;
  ap.scale = pair->scale;
  ap.ret_count = pair->ret_count;
  ap.ret_offset = pair->ret_offset;
  ap.ret_index = pair->ret_index;
  ap.ret_rows = (const char*)pair->ret_rows;
  ap.q = (const char*)q;
  ap.k_new = (const char*)k_new;
  ap.v_new = (const char*)v_new;
  ap.status = pair->status;
  ap.scale_log2 = sm_scale * 1.44269504088896340736f;
  ap.layer_sel = layer_sel == MC_LAYER_BOTH ? 0 : layer_sel;
  ap.n_sets = layer_sel == MC_LAYER_BOTH ? 2 : 1;
  ap.nq = cfg->n_q_heads / cfg->n_kv_heads;
  ap.rows = ap.n_sets * ap.nq;
  ap.n_q_heads = cfg->n_q_heads;
  ap.split_len = pick_split_len(cfg, bt);
  ap.n_splits = max(1, (bt->max_seq_len + ap.split_len - 1) / ap.split_len);
  const size_t prow = (size_t)ap.n_sets * bt->batch * cfg->n_q_heads * ap.n_splits;
  ap.part_o = reinterpret_cast<float*>(workspace);
  ap.part_ml = reinterpret_cast<float*>((char*)workspace + align_up(prow * kHeadDim * 4, 256));

  CUtensorMap tm_k, tm_v;
  const int64_t n_rows = bt->n_pages * cfg->n_kv_heads * cfg->page_size;
  mc_status st = encode_pool_map(&tm_k, pair->e_k, cfg->dtype, n_rows, cfg->page_size);
  if (st != MC_OK) return st;
  st = encode_pool_map(&tm_v, pair->e_v, cfg->dtype, n_rows, cfg->page_size);
  if (st != MC_OK) return st;

  const size_t smem = attn_smem_bytes(ap.split_len);
  dim3 grid(ap.n_splits, cfg->n_kv_heads, bt->batch);
  dim3 cgrid(cfg->n_q_heads, bt->batch, ap.n_sets);
  if (cfg->dtype == MC_F16) {
    MC_CUDA_CHECK(cudaFuncSetAttribute(attn_split_kernel<MC_F16>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem));
    attn_split_kernel<MC_F16><<<grid, kAttnThreads, smem, stream>>>(tm_k, tm_v, ap);
    MC_CUDA_CHECK(cudaGetLastError());
    attn_combine_kernel<MC_F16><<<cgrid, 128, 0, stream>>>(ap, (unsigned short*)out, lse);
  } else {
    MC_CUDA_CHECK(cudaFuncSetAttribute(attn_split_kernel<MC_BF16>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem));
    attn_split_kernel<MC_BF16><<<grid, kAttnThreads, smem, stream>>>(tm_k, tm_v, ap);
    MC_CUDA_CHECK(cudaGetLastError());
    attn_combine_kernel<MC_BF16><<<cgrid, 128, 0, stream>>>(ap, (unsigned short*)out, lse);
  }
  MC_CUDA_CHECK(cudaGetLastError());
  return MC_OK;
}

}  // namespace mc

// ---------------------------------------------------------------------------------------------------
// Decode attention for callers that cannot supply scratch memory: the split partials live in a
// device array that is part of the library image.
// ---------------------------------------------------------------------------------------------------
#include <mutex>
#include <stdio.h>

static __device__ __align__(256) unsigned char g_static_scratch[MC_STATIC_SCRATCH_BYTES];

namespace {
constexpr int kMaxDevices = 64;
std::mutex g_scratch_mutex;
void* g_scratch_addr[kMaxDevices] = {nullptr};  // device address of g_static_scratch, per device
}  // namespace

extern "C" mc_status mc_decode_attn_static(const mc_config* cfg, const mc_batch* batch, const mc_pair_cache* pair,
                                           int32_t layer_sel, const void* q, const void* k_new, const void* v_new,
                                           float sm_scale, void* out, float* lse, void* stream) {
  if (layer_sel < MC_LAYER_LM1 || layer_sel > MC_LAYER_BOTH) return MC_ERR_INVALID_ARG;
  const int n_sets = layer_sel == MC_LAYER_BOTH ? 2 : 1;
  size_t need = 0;
  const mc_status st = mc_workspace_bytes(cfg, batch, MC_OP_DECODE_ATTN, n_sets, &need);  // validates cfg, host only
  if (st != MC_OK) return st;
  if (need > (size_t)MC_STATIC_SCRATCH_BYTES) {
    char msg[160];
    snprintf(msg, sizeof(msg), "mc_decode_attn_static: partials need %zu bytes, built-in scratch holds %u", need,
             (unsigned)MC_STATIC_SCRATCH_BYTES);
    mc::set_cuda_error(cudaSuccess, msg);
    return MC_ERR_CAPACITY;
  }
  int dev = -1;
  MC_CUDA_CHECK(cudaGetDevice(&dev));
  if (dev < 0 || dev >= kMaxDevices) return MC_ERR_UNSUPPORTED;
  void* scratch = nullptr;
  {
    std::lock_guard<std::mutex> lock(g_scratch_mutex);
    if (g_scratch_addr[dev] == nullptr) {
      // In host code `g_static_scratch` is only a handle for the symbol; the address the kernels
      // must be given comes from the runtime, separately for each device.
      void* ptr = nullptr;
      MC_CUDA_CHECK(cudaGetSymbolAddress(&ptr, g_static_scratch));
      g_scratch_addr[dev] = ptr;
    }
    scratch = g_scratch_addr[dev];
  }
  return mc_decode_attn(cfg, batch, pair, layer_sel, q, k_new, v_new, sm_scale, out, lse, scratch,
                        (size_t)MC_STATIC_SCRATCH_BYTES, stream);
}
