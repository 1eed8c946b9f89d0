// Single-query decode attention straight over the compressed pair cache
// (Algorithm 2 "MiniCache Decoding": rescale by the layer's magnitude, put the retained rows
// back, append the new token, softmax(q K^T) V), with the restore folded into the kernel:
//
//   q . (g_i e_i) = g_i (q . e_i)              the K scale multiplies the score
//   sum_i p_i (g_i e_i) = sum_i (p_i g_i) e_i  the V scale multiplies the probability
//
// so the shared direction rows are streamed once, untouched; a retained token (whose scales the
// merge left at -0) only replaces one score (K) or adds one term to the sum (V).
//
// The kernel is persistent, two CTAs per SM.  The token axis is cut into equal shares for teams of
// CTAs, a team member takes its team's share for one kv head (see piece_at); a work item
// is a chunk of a piece: a run of 128-token units of one (sequence, kv head).  In each CTA
//   - the producer warp streams everything a piece needs through one ring of stages with bulk
//     asynchronous copies (TMA engine, cp.async.bulk + mbarrier): one copy per (page, head, tensor)
//     tile, all K tiles of the piece, then "extra" stages holding the piece's retained K rows and
//     the step's new K row, then the V tiles and the V extras; it runs ahead into the next piece,
//     and loads page ids and retained ranges one piece early (a demand load takes microseconds
//     while the copy engine saturates the memory system, so nothing irregular is left on any
//     critical path);
//   - four consumer warps run every contraction on the tensor cores, the query rows of the kv
//     head's group (and of both layers in pair mode) being the 8-wide N tile and the cached rows
//     the M tile: scores x K scale -> shared memory (the scores of retained rows, from their raw
//     rows, fill the columns the tiles leave out), row maxima tracked on the way -> V phase: each
//     warp takes 16 tokens of every tile, P = 2^(score - max) x V scale formed where it is used,
//     plus gathered P times the retained V rows; the warps' partial sums meet in shared memory.
// Partial (m, l, o) per piece are merged by attn_combine_kernel.  Every wait is bounded.
#include <string.h>

#include <algorithm>

#include "mc_common.cuh"
#include "mc_kernels.h"
#include "mc_pipe.cuh"
#include "mc_q4.cuh"
#include "mc_append.cuh"

namespace mc {

constexpr int kTile = 64;  // tokens per pipeline stage
constexpr int kUnit_ = 128;  // (= kUnit below) tokens per stage of 4-bit tiles
constexpr int kStages = 5;      // ring stages of the 16-bit kernel with one query row per kv head
constexpr int kStagesWide = 4;  // ... with several rows: a stage is given up for a score buffer twice the size
constexpr int kConsumerWarps = 4;
constexpr int kConsumerThreads = kConsumerWarps * 32;
constexpr int kAttnThreads = kConsumerThreads + 32;  // + producer warp
constexpr int kMaxRows = 8;                          // query rows per (sequence, kv head): the 8-wide N tile
constexpr int kStageBytes = (kTile / 16) * (16 * kRowBytes + 2 * 16 * 4);  // 64 tokens of tiles: 16896 for any page size
constexpr int kQ4StageBytes = (kUnit_ / kQ4Page) * kQ4TileBytes;  // four 4-bit tiles: 11264
constexpr int kQ4Stages = 5;
constexpr int kEntryBytes = 272;  // a retained entry: 256-byte raw row, int32 token index, padding
constexpr int kMaxBatchSmem = 512;
constexpr int kCtasPerSm = 2;
constexpr int kSlabStride = 132;  // floats per row of a warp's partial output in shared memory (4 mod 32: no bank conflicts)

struct AttnParams {
  Geom g;
  const char* e_pool[2];  // compressed tiles: K, V
  const char* res_pool[2];  // 4-bit cache: the residual 16-bit tiles [batch][H][kResTileBytes]
  const int32_t* ret_offset;
  const int32_t* ret_prefix;
  int ret_prefix_stride;
  const char* ret_rows;  // [2 layers][ret_capacity][kEntryBytes]
  int64_t ret_capacity;
  const char* q;
  const char* k_new;
  const char* v_new;
  float* part_o;   // [n_sets][batch][Hq][slots][128]: a piece's partial sits in the slot of its first unit
  float* part_ml;  // [n_sets][batch][Hq][slots][2]
  int32_t* status;
  float scale_log2;  // sm_scale * log2(e)
  int layer_sel;
  int n_sets;
  int nq;    // query heads per kv head
  int rows;  // n_sets * nq
  int n_q_heads;
  int cap_units;  // longest chunk, in units of 128 tokens (what the score buffer holds for `rows` rows)
  int slots;      // partial slots per output row = units of the longest sequence
  int team_size;  // CTAs per team (one or more kv heads each)
  int n_teams;
};

// ---- PTX wrappers (tensor-core side; the copy/barrier wrappers live in mc_pipe.cuh) ---------------
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
// D += A(16x16, rows 8..15 zero) * B(16x8); only the accumulator registers of rows 0..7 matter.
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
// D(16x8) += A(16x16) * B(16x8), all of A used: the cached rows are the A operand (16 tokens x 16
// channels for the scores, 16 channels x 16 tokens for the output), the query rows / probabilities
// the 8-wide B operand, so that every accumulator register holds a wanted number.
template <int DT>
__device__ __forceinline__ void mma_rows(float (&c)[4], uint32_t a0, uint32_t a1, uint32_t a2, uint32_t a3, uint32_t b0,
                                         uint32_t b1) {
  if (DT == MC_F16) {
    asm volatile(
        "mma.sync.aligned.m16n8k16.row.col.f32.f16.f16.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%0,%1,%2,%3};"
        : "+f"(c[0]), "+f"(c[1]), "+f"(c[2]), "+f"(c[3])
        : "r"(a0), "r"(a1), "r"(a2), "r"(a3), "r"(b0), "r"(b1));
  } else {
    asm volatile(
        "mma.sync.aligned.m16n8k16.row.col.f32.bf16.bf16.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%0,%1,%2,%3};"
        : "+f"(c[0]), "+f"(c[1]), "+f"(c[2]), "+f"(c[3])
        : "r"(a0), "r"(a1), "r"(a2), "r"(a3), "r"(b0), "r"(b1));
  }
}
__device__ __forceinline__ void consumer_sync() { asm volatile("bar.sync 1, %0;" ::"n"(kConsumerThreads) : "memory"); }

// Shared-memory address of 16-byte chunk `chunk` (0..15) of token row `tk` (0..63) of a stage.
// A stage holds 64 / page_size tiles back to back, each as in global memory (see tile_bytes).
__device__ __forceinline__ uint32_t tile_addr(uint32_t stage, int tk, int chunk, int page_shift, int tbytes) {
  const int j = tk >> page_shift;
  const int r = tk & ((1 << page_shift) - 1);
  return stage + (uint32_t)(j * tbytes + r * kRowBytes + (chunk_pos(r, chunk) << 4));
}

constexpr int kUnit = 128;            // tokens per unit of work: pieces start and end on unit boundaries
// Floats of the score buffer S [rows][piece tokens + 8]: 16.5 KB, or 33 KB (WIDE) where several query rows share
// a kv head (grouped queries, pair mode) and for the 4-bit cache, whose stages are smaller: chunks twice as long,
// half as many switches between the K and the V phase of a piece.
constexpr int kScoreFloats = 4224;
constexpr int kScoreFloatsWide = 8448;
constexpr int kMaxPiecePages = 256;   // pages of the longest piece (4096 tokens of 16-token pages)

// Longest chunk for `rows` query rows: rows x (tokens + 8) floats must fit the score buffer.
__host__ __device__ __forceinline__ int piece_cap_units(int rows, bool wide) {
  const int u = ((wide ? kScoreFloatsWide : kScoreFloats) / rows - 8) / kUnit;
  return u > 32 ? 32 : u;  // 32 units (rows = 1) ... 4 units (rows = 8; 8 with the wide buffer)
}
// The same memory later holds the four warps' partial outputs [4][rows][kSlabStride].
static_assert(kMaxRows * ((kScoreFloats / kMaxRows - 8) / kUnit * kUnit + 8) <= kScoreFloats, "score buffer");
static_assert(kMaxRows * ((kScoreFloatsWide / kMaxRows - 8) / kUnit * kUnit + 8) <= kScoreFloatsWide, "score buffer");
static_assert(kConsumerWarps * kMaxRows * kSlabStride <= kScoreFloats, "slabs fit the score buffer");

// The merge marks a retained token by the scale -0: the shared direction then contributes nothing
// wherever scales are applied blindly, and a token whose rows are genuinely zero (scale +0, score 0)
// stays distinguishable.
__device__ __forceinline__ bool is_retained_scale(float g) { return __float_as_uint(g) == 0x80000000u; }

// One work item = a chunk of a piece: a run of units of one (sequence, kv head).
struct Item {
  int b, g, split;  // split = the piece's first unit inside its sequence (its partial slot)
  int split_start;  // first token of this chunk
  int n_tok;    // cached tokens of this chunk
  int T;        // 64-token tiles
  int n_q;      // 4-bit cache: tokens of this chunk that live in 4-bit pages (a multiple of 32; the rest,
                // at most 31 at the sequence's end, sit in the residual tile)
  int Tq;       // 4-bit cache: stages of up to four 4-bit pages (128 tokens)
  int TT;       // tile stages of a phase: T, or Tq plus one for the residual tile
  int units;
  bool first, last;  // first / last chunk of its piece
  bool has_new;
  bool valid;
};

// Work is cut along the token axis only.  A sequence owns max(1, ceil(n / 128)) units (pre_s =
// exclusive prefix over sequences, U units in all).  The grid is T teams of S CTAs: team t takes
// the units [t U / T, (t + 1) U / T) -- the same share for every team whatever the lengths are --
// and its member j takes them for the kv heads j, j + S, ...  The members of a team stream the
// same pages at about the same time (neighbouring tiles of a page: whole DRAM rows get used), and
// nobody waits for a last round of items.  A piece = the units of one (sequence, head) inside a
// team's range: one partial result.  A CTA works through a piece in chunks of as many units as the
// score buffer holds, carrying the running maximum, sum and output from chunk to chunk.
struct Cursor {
  int g, x;  // kv head, unit
};
template <bool Q4>
__device__ __forceinline__ Item piece_at(const Cursor& c, int x_begin, int x_end, const int* pre_s, const int* len_s,
                                         const AttnParams& p) {
  Item it;
  it.valid = c.g < p.g.n_kv_heads && c.x < x_end;
  if (!it.valid) {
    it.b = it.g = it.split = it.split_start = it.n_tok = it.T = it.units = it.n_q = it.Tq = it.TT = 0;
    it.has_new = it.first = it.last = false;
    return it;
  }
  int lo = 0, hi = p.g.batch - 1;  // last b with pre_s[b] <= x
  while (lo < hi) {
    const int mid = (lo + hi + 1) >> 1;
    if (pre_s[mid] <= c.x) lo = mid; else hi = mid - 1;
  }
  it.b = lo;
  it.g = c.g;
  const int u_b = pre_s[lo + 1] - pre_s[lo];
  const int k = c.x - pre_s[lo];                        // this chunk's first unit inside the sequence
  const int k_lo = max(0, x_begin - pre_s[lo]);         // the piece's first unit
  const int k_hi = min(u_b, x_end - pre_s[lo]);         // one past the piece's last unit
  it.split = k_lo;
  it.units = min(k_hi - k, p.cap_units);
  it.first = k == k_lo;
  it.last = k + it.units == k_hi;
  const int n = len_s[lo];
  it.split_start = k * kUnit;
  it.n_tok = max(0, min(n, (k + it.units) * kUnit) - it.split_start);
  it.T = (it.n_tok + kTile - 1) / kTile;
  it.n_q = Q4 ? max(0, min(it.n_tok, (n & ~(kQ4Page - 1)) - it.split_start)) : 0;
  it.Tq = (it.n_q + kUnit - 1) / kUnit;
  it.TT = Q4 ? it.Tq + (it.n_tok > it.n_q ? 1 : 0) : it.T;
  it.has_new = (p.k_new != nullptr) && (k + it.units == u_b);
  return it;
}
// The cursor after piece `it`: on through the team's range, then the member's next head.
__device__ __forceinline__ Cursor next_cursor(const Cursor& c, const Item& it, int x_begin, int x_end, int team_size) {
  Cursor n = c;
  n.x += it.units;
  if (n.x >= x_end) {
    n.x = x_begin;
    n.g += team_size;
  }
  return n;
}

// Where an item's retained entries sit in the pair's lists (first entry, count) for K and V.
struct Ranges {
  int k_lo, n_k, v_lo, n_v;
};

// Two table entries per list: piece boundaries are multiples of 128 and no retained token lies
// past the length the pair was merged at.  The loads are issued one item ahead and only combined
// (ranges_of) when that item starts: arithmetic on a loaded value would stall the producer warp for
// the load's whole latency, microseconds while the copy engine saturates the memory system.
struct RawRanges {
  int off_k, off_v, k0, k1, v0, v1;
};
__device__ __forceinline__ RawRanges load_ranges(const Item& w, const AttnParams& p) {
  RawRanges r;
  r.off_k = r.off_v = r.k0 = r.k1 = r.v0 = r.v1 = 0;
  // (an empty sequence has no retained tokens; its tables may be being rewritten by an admission)
  if (!w.valid || w.n_tok == 0) return r;
  const int H = p.g.n_kv_heads;
  const int seg_k = w.b * H + w.g, seg_v = (p.g.batch + w.b) * H + w.g;
  const int pj0 = min(w.split_start >> 7, p.ret_prefix_stride - 1);
  const int pj1 = min((w.split_start + w.n_tok + 127) >> 7, p.ret_prefix_stride - 1);
  const int32_t* pk = p.ret_prefix + (size_t)seg_k * p.ret_prefix_stride;
  const int32_t* pv = p.ret_prefix + (size_t)seg_v * p.ret_prefix_stride;
  r.off_k = __ldg(p.ret_offset + seg_k);
  r.off_v = __ldg(p.ret_offset + seg_v);
  r.k0 = __ldg(pk + pj0);
  r.k1 = __ldg(pk + pj1);
  r.v0 = __ldg(pv + pj0);
  r.v1 = __ldg(pv + pj1);
  return r;
}
__device__ __forceinline__ Ranges ranges_of(const RawRanges& q) {
  Ranges r;
  r.k_lo = q.off_k + q.k0;
  r.n_k = q.k1 - q.k0;
  r.v_lo = q.off_v + q.v0;
  r.n_v = q.v1 - q.v0;
  return r;
}

// Q4: the pair is a 4-bit shared cache (pages of 32 tokens): a tile stage holds up to four 4-bit tiles
// (128 tokens, one page per consumer warp), whose tensor-core fragments are built in registers straight
// from the codes (code * scale + zero in one packed 16-bit FMA, the exact stored direction); the tokens
// of a sequence's last, incomplete page arrive as one more tile stage in the 16-bit format.
template <int DT, bool Q4, bool WIDE>
__global__ void __launch_bounds__(kAttnThreads, kCtasPerSm) attn_split_kernel(const AttnParams p) {
  // The batch description (lengths, block table) and the queries belong to the caller: no kernel of
  // this library writes them, so they are read before the wait on the previous kernel in the
  // stream (whose tail this prologue then overlaps).  The pair cache and the workspace are touched
  // only after the wait.
  // stage ring: five slots of 64 tokens of 16-bit tiles, or (4-bit cache) four slots of four 4-bit tiles,
  // which also hold the residual tile or a stage of retained entries
  constexpr int STAGE_BYTES = Q4 ? kQ4StageBytes : kStageBytes;
  constexpr int N_STAGES = Q4 ? kQ4Stages : (WIDE ? kStagesWide : kStages);
  constexpr int SCORE_FLOATS = WIDE ? kScoreFloatsWide : kScoreFloats;
  grid_dep_launch();
  const int ps = p.g.page_size, shift = p.g.page_shift;
  const int H = p.g.n_kv_heads;
  const int tbytes = tile_bytes(ps);
  const int nslots = p.n_sets;
  const int rows = p.rows;
  const int s_stride = p.cap_units * kUnit + 8;
  const int cap_e = nslots == 2 ? 16 : 32;  // retained entries (per layer) in one extra stage
  const int set_bytes = cap_e * kEntryBytes;

  extern __shared__ unsigned char smem_raw[];
  unsigned char* smem = reinterpret_cast<unsigned char*>((reinterpret_cast<uintptr_t>(smem_raw) + 127) & ~uintptr_t(127));
  unsigned char* stages = smem;
  float* S = reinterpret_cast<float*>(smem + N_STAGES * STAGE_BYTES);     // [kMaxRows][s_stride]
  uint32_t* q_s = reinterpret_cast<uint32_t*>(S + SCORE_FLOATS);         // [2][kMaxRows][64] packed pairs
  float* m_s = reinterpret_cast<float*>(q_s + 2 * kMaxRows * 64);        // [kMaxRows]
  float* l_s = m_s + kMaxRows;                                           // [kMaxRows][kConsumerWarps]
  float* red_s = l_s + kMaxRows * kConsumerWarps;                        // [kMaxRows][kConsumerWarps]
  float* red2_s = red_s + kMaxRows * kConsumerWarps;                     // [kMaxRows][kConsumerWarps]
  int* info_s = reinterpret_cast<int*>(red2_s + kMaxRows * kConsumerWarps);  // [N_STAGES][2]: entries, extra stages of the phase
  int* pre_s = info_s + 2 * N_STAGES;                                     // [batch + 1] unit-count prefix
  int* len_s = pre_s + kMaxBatchSmem + 1;                                // [batch] sequence lengths
  int* pages_s = len_s + kMaxBatchSmem;                                  // [2][kMaxPiecePages] page ids of a piece
  volatile int* s_abort = pages_s + 2 * kMaxPiecePages;
  uint64_t* bars = reinterpret_cast<uint64_t*>((reinterpret_cast<uintptr_t>(s_abort + 1) + 7) & ~uintptr_t(7));
  const uint32_t full0 = smem_u32(bars), empty0 = full0 + 8 * N_STAGES;
  const uint32_t stage0 = smem_u32(stages);

  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;

  // ---- prologue -----------------------------------------------------------------------------------
  if (tid == 0) {
    for (int s = 0; s < N_STAGES; ++s) {
      mbar_init(full0 + 8 * s, 1);
      mbar_init(empty0 + 8 * s, kConsumerWarps);
    }
    *s_abort = 0;
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  // (a length above the declared bound is clamped here, so that a sequence never owns more units than
  // it has partial slots, and flagged once the status words may be touched)
  int bad_meta = 0;
  for (int b = tid; b < p.g.batch; b += kAttnThreads) {
    const int n = p.g.seq_lens[b];
    bad_meta |= (n < 0 || n > p.g.max_seq_len) ? 1 : 0;
    len_s[b] = min(max(n, 0), p.g.max_seq_len);
  }
  __syncthreads();
  if (tid == 0) {
    // prefix of the sequences' unit counts (a sequence always owns at least one unit)
    int acc = 0;
    for (int b = 0; b < p.g.batch; ++b) {
      pre_s[b] = acc;
      acc += max(1, (len_s[b] + kUnit - 1) / kUnit);
    }
    pre_s[p.g.batch] = acc;
  }
  __syncthreads();
  const int n_teams = p.n_teams;
  const int team = blockIdx.x / p.team_size;
  const long long n_units = pre_s[p.g.batch];
  const int x_begin = (int)(n_units * team / n_teams), x_end = (int)(n_units * (team + 1) / n_teams);
  const Cursor c_first = {(int)(blockIdx.x % p.team_size), x_begin};

  if (warp == kConsumerWarps) {
    // ===================== producer =====================
    // Everything an item needs from global memory before its copies can be issued (page ids,
    // retained ranges) is loaded one item ahead: such loads take microseconds while the copy
    // engine saturates the memory system.
    int it = 0;  // running stage counter, same sequence as the consumers'
    Cursor cur = c_first;
    Item w = piece_at<Q4>(cur, x_begin, x_end, pre_s, len_s, p);
    RawRanges raw;
    // page ids of a piece: lane l holds pages l, l + 32, ... (registers, loaded one piece ahead),
    // handed over to shared memory when the piece starts
    int pg_reg[kMaxPiecePages / 32];
    auto load_pages = [&](const Item& it) {
      const int np = (it.n_tok + ps - 1) >> shift;
      const int32_t* row = p.g.block_table + (size_t)it.b * p.g.max_pages_per_seq + (it.split_start >> shift);
#pragma unroll
      for (int r = 0; r < kMaxPiecePages / 32; ++r) {
        pg_reg[r] = 0;
        if (it.valid && lane + 32 * r < np) pg_reg[r] = row[lane + 32 * r];
        // a page id outside the pools never becomes a copy's source address: page 0 is streamed
        // instead and the call is flagged (its result for that sequence means nothing)
        if (!page_ok(p.g, pg_reg[r])) {
          pg_reg[r] = 0;
          bad_meta = 1;
        }
      }
    };
    load_pages(w);
    grid_dep_wait();
    if (bad_meta) {
      atomicOr(p.status, MC_FLAG_BAD_METADATA);
      bad_meta = 0;
    }
    raw = load_ranges(w, p);
    bool ok = true;
    int n_piece = 0;
    for (; w.valid && ok; ++n_piece) {
      int* pages = pages_s + (n_piece & 1) * kMaxPiecePages;
#pragma unroll
      for (int r = 0; r < kMaxPiecePages / 32; ++r) pages[lane + 32 * r] = pg_reg[r];
      __syncwarp();
      cur = next_cursor(cur, w, x_begin, x_end, p.team_size);
      const Item wn = piece_at<Q4>(cur, x_begin, x_end, pre_s, len_s, p);
      const RawRanges rawn = load_ranges(wn, p);
      load_pages(wn);
      if (bad_meta) {
        atomicOr(p.status, MC_FLAG_BAD_METADATA);
        bad_meta = 0;
      }
      const int n_pages_item = (w.n_tok + ps - 1) >> shift;
      const int n_new = w.has_new ? 1 : 0;
      for (int ph = 0; ph < 2 && ok; ++ph) {
        // The retained ranges (loaded one piece ago; for a CTA's first piece just now) are looked at
        // only when the last tile goes out: the consumers take the number of extra stages from the
        // last tile's stage, so the tiles before it need not wait for those loads.
        int n_r = 0, r_lo = 0;
        int X = -1;  // extra stages: retained rows and the new token
        for (int t = 0;; ++t, ++it) {
          if (X < 0 && t >= w.TT - 1) {
            const Ranges rg = ranges_of(raw);
            n_r = ph ? rg.n_v : rg.n_k;
            r_lo = ph ? rg.v_lo : rg.k_lo;
            // (range-checked build: a retained range that does not fit the pool or the chunk is not followed)
            if (!MC_IN_BOUNDS(n_r >= 0 && r_lo >= 0 && n_r <= w.n_tok && (int64_t)r_lo + n_r <= p.ret_capacity, p.status)) n_r = 0;
            X = (n_r + n_new + cap_e - 1) / cap_e;
          }
          if (X >= 0 && t >= w.TT + X) break;
          const int s = it % N_STAGES;
          if (it >= N_STAGES) {
            int good = 1;
            if (lane == 0) good = mbar_wait(empty0 + 8 * s, ((it / N_STAGES) - 1) & 1, s_abort, p.status) ? 1 : 0;
            good = __shfl_sync(0xffffffffu, good, 0);
            if (!good) { ok = false; break; }
          }
          const uint32_t bar = full0 + 8 * s;
          const uint32_t sbase = stage0 + s * STAGE_BYTES;
          if (Q4 && t < w.Tq) {
            // ---- up to four 4-bit pages (128 tokens): a bulk copy per page
            const int n_pg = min(kUnit / kQ4Page, (w.n_q >> 5) - t * (kUnit / kQ4Page));
            if (lane == 0) {
              info_s[2 * s] = 0;
              info_s[2 * s + 1] = X;
              mbar_expect_tx(bar, (uint32_t)(n_pg * kQ4TileBytes));
            }
            __syncwarp();
            if (lane < n_pg)
              bulk_load(sbase + lane * kQ4TileBytes,
                        p.e_pool[ph] + ((size_t)pages[t * (kUnit / kQ4Page) + lane] * H + w.g) * kQ4TileBytes,
                        (uint32_t)kQ4TileBytes, bar);
          } else if (Q4 && t < w.TT) {
            // ---- the residual tile: the sequence's last, incomplete page in 16 bits
            if (lane == 0) {
              info_s[2 * s] = 0;
              info_s[2 * s + 1] = X;
              mbar_expect_tx(bar, (uint32_t)kResTileBytes);
              bulk_load(sbase, p.res_pool[ph] + ((size_t)w.b * H + w.g) * kResTileBytes, (uint32_t)kResTileBytes, bar);
            }
            __syncwarp();
          } else if (t < w.TT) {
            // ---- one 64-token tile: a bulk copy per page
            const int pg0 = (t * kTile) >> shift;
            const int n_pg = min(kTile >> shift, n_pages_item - pg0);
            if (lane == 0) {
              info_s[2 * s] = 0;
              info_s[2 * s + 1] = X;
              mbar_expect_tx(bar, (uint32_t)(n_pg * tbytes));
            }
            __syncwarp();
            if (lane < n_pg)
              bulk_load(sbase + lane * tbytes, p.e_pool[ph] + ((size_t)pages[pg0 + lane] * H + w.g) * tbytes, (uint32_t)tbytes,
                        bar);
          } else {
            // ---- an extra stage: up to cap_e retained entries per layer, the new token last
            const int x0 = (t - w.TT) * cap_e;
            const int cnt_ret = max(0, min(n_r, x0 + cap_e) - x0);
            const bool add_new = n_new && n_r >= x0 && n_r < x0 + cap_e;
            if (lane == 0) {
              info_s[2 * s] = cnt_ret + (add_new ? 1 : 0);
              info_s[2 * s + 1] = X;
              if (add_new) {
                for (int set = 0; set < nslots; ++set)
                  *reinterpret_cast<int*>(stages + s * STAGE_BYTES + set * set_bytes + cnt_ret * kEntryBytes + kRowBytes) =
                      w.split_start + w.n_tok;  // the new token's index
              }
              mbar_expect_tx(bar, (uint32_t)(nslots * (cnt_ret * kEntryBytes + (add_new ? kRowBytes : 0))));
            }
            __syncwarp();
            if (lane < nslots && cnt_ret > 0) {
              const int layer = nslots == 2 ? lane : p.layer_sel;
              bulk_load(sbase + lane * set_bytes, p.ret_rows + ((size_t)layer * p.ret_capacity + r_lo + x0) * kEntryBytes,
                        (uint32_t)(cnt_ret * kEntryBytes), bar);
            }
            if (lane >= 2 && lane < 2 + nslots && add_new) {
              const int set = lane - 2;
              const char* src = (ph ? p.v_new : p.k_new) + (((size_t)set * p.g.batch + w.b) * H + w.g) * kRowBytes;
              bulk_load(sbase + set * set_bytes + cnt_ret * kEntryBytes, src, (uint32_t)kRowBytes, bar);
            }
          }
        }
      }
      w = wn;
      raw = rawn;
    }
    return;
  }

  // ===================== consumers =====================
  const int row = lane >> 2;        // M-tile row of this thread's fragments
  const int colp = (lane & 3) * 2;  // column pair inside an 8-wide n tile
  const int set_row = (nslots == 2 && row < rows) ? row / p.nq : 0;  // which layer this row attends (pair mode)
  const int slot_row = nslots == 2 ? set_row : p.layer_sel;          // which of the tile's two scales it uses
  const int mi = lane >> 3, mr = lane & 7;
  // the two query rows whose results this thread holds when the rows are the n dimension
  const int slot0 = nslots == 2 ? min(colp / p.nq, 1) : p.layer_sel;
  const int slot1 = nslots == 2 ? min((colp + 1) / p.nq, 1) : p.layer_sel;
  int it = 0, n_item = 0;

  auto load_q_words = [&](const Item& w, uint32_t (&qw)[4]) {
#pragma unroll
    for (int k = 0; k < 4; ++k) {
      const int i = tid + k * kConsumerThreads;  // 512 words = 8 rows x 64
      const int r = i >> 6, wd = i & 63;
      uint32_t v = 0;
      if (w.valid && r < rows) {
        const int set = r / p.nq, rq = r - set * p.nq;
        const size_t qrow = ((size_t)set * p.g.batch + w.b) * p.n_q_heads + w.g * p.nq + rq;
        v = reinterpret_cast<const uint32_t*>(p.q)[qrow * 64 + wd];
      }
      qw[k] = v;
    }
  };
  {
    uint32_t qw[4];
    load_q_words(piece_at<Q4>(c_first, x_begin, x_end, pre_s, len_s, p), qw);
#pragma unroll
    for (int k = 0; k < 4; ++k) q_s[tid + k * kConsumerThreads] = qw[k];
  }
  grid_dep_wait();
  if (bad_meta) atomicOr(p.status, MC_FLAG_BAD_METADATA);
  consumer_sync();

  // carried from chunk to chunk of a piece: the output sums, this thread's part of the row sum, and
  // the running maxima of the rows this thread meets (row `row` in the V phase, rows colp and
  // colp + 1 in its accumulators)
  float acc[8][4];
  float l_acc = 0.f, m_run = -INFINITY, m_run0 = -INFINITY, m_run1 = -INFINITY;
  Cursor cur = c_first;
  for (;; ++n_item) {
    const Item w = piece_at<Q4>(cur, x_begin, x_end, pre_s, len_s, p);
    if (!w.valid) break;
    cur = next_cursor(cur, w, x_begin, x_end, p.team_size);
    const uint32_t* qcur = q_s + (n_item & 1) * kMaxRows * 64;
    const int n_new = w.has_new ? 1 : 0;
    bool ok = true;

    float mx0 = -INFINITY, mx1 = -INFINITY, mxe = -INFINITY;  // running maxima of the scores this thread stores
    // ---- K phase: S[r][i] = log2e * sm_scale * g_i * (q_r . e_i) ---------------------------------
    {
      // query fragments for 16-bit rows (k step ks: channels 16 ks + 2 t4 + {0, 1} and + {8, 9}); with a
      // 4-bit cache they are fetched only where a 16-bit stage needs them (residual tile, raw rows)
      uint32_t qa0[8], qa2[8];
      auto load_qa = [&]() {
#pragma unroll
        for (int ks = 0; ks < 8; ++ks) {
          qa0[ks] = qcur[row * 64 + ks * 8 + (lane & 3)];
          qa2[ks] = qcur[row * 64 + ks * 8 + 4 + (lane & 3)];
        }
      };
      if (!Q4) load_qa();
      // 4-bit tiles: lane (row, t4) owns the channels [32 t4, 32 t4 + 32) of its token rows (16 bytes of
      // codes); k step ks pairs the channels 32 t4 + 4 ks + {0, 1} and + {2, 3} with the matching query words
      uint32_t qk0[8], qk2[8];
      if (Q4) {
#pragma unroll
        for (int ks = 0; ks < 8; ++ks) {
          qk0[ks] = qcur[row * 64 + 16 * (lane & 3) + 2 * ks];
          qk2[ks] = qcur[row * 64 + 16 * (lane & 3) + 2 * ks + 1];
        }
      }
      const int tk_w = warp * 16;  // this warp's 16 tokens of every tile
      int xk = n_new;              // extra stages after the tiles (an item without tiles has no retained rows)
      for (int t = 0; t < w.TT; ++t, ++it) {
        const int s = it % N_STAGES;
        if (!mbar_wait(full0 + 8 * s, (it / N_STAGES) & 1, s_abort, p.status)) { ok = false; break; }
        const uint32_t sbase = stage0 + s * STAGE_BYTES;
        xk = info_s[2 * s + 1];
        if (Q4 && t < w.Tq) {
          // ---- four 4-bit pages, one per warp
          if (warp < (w.n_q >> 5) - t * (kUnit / kQ4Page)) {
            const unsigned char* tb = stages + s * STAGE_BYTES + warp * kQ4TileBytes;
            const int t4 = lane & 3;
            uint4 sK[4], zK[4];  // the group parameters of this lane's 32 channels, word k = channels 8 (4 t4 + k) + ...
#pragma unroll
            for (int k = 0; k < 4; ++k) {
              sK[k] = *reinterpret_cast<const uint4*>(tb + kQ4CodeBytes + (4 * k + t4) * 16);
              zK[k] = *reinterpret_cast<const uint4*>(tb + kQ4CodeBytes + 256 + (4 * k + t4) * 16);
            }
            const float* gq = reinterpret_cast<const float*>(tb + kQ4ScaleOff);
#pragma unroll
            for (int hf = 0; hf < 2; ++hf) {
              const int ra_ = 16 * hf + row;  // this lane's token rows inside the page: ra_, ra_ + 8
              const uint4 wA = *reinterpret_cast<const uint4*>(tb + ra_ * 64 + t4 * 16);
              const uint4 wB = *reinterpret_cast<const uint4*>(tb + (ra_ + 8) * 64 + t4 * 16);
              const uint32_t wa[4] = {wA.x, wA.y, wA.z, wA.w}, wb[4] = {wB.x, wB.y, wB.z, wB.w};
              float acc0[4] = {0.f, 0.f, 0.f, 0.f}, acc1[4] = {0.f, 0.f, 0.f, 0.f};
#pragma unroll
              for (int k = 0; k < 4; ++k) {
                uint32_t cA[4], cB[4];
                code_pairs<DT>(wa[k], cA);
                code_pairs<DT>(wb[k], cB);
                const uint32_t sk[4] = {sK[k].x, sK[k].y, sK[k].z, sK[k].w}, zk[4] = {zK[k].x, zK[k].y, zK[k].z, zK[k].w};
                mma_rows<DT>(acc0, deq_pair<DT>(cA[0], sk[0], zk[0]), deq_pair<DT>(cB[0], sk[0], zk[0]),
                             deq_pair<DT>(cA[1], sk[1], zk[1]), deq_pair<DT>(cB[1], sk[1], zk[1]), qk0[2 * k], qk2[2 * k]);
                mma_rows<DT>(acc1, deq_pair<DT>(cA[2], sk[2], zk[2]), deq_pair<DT>(cB[2], sk[2], zk[2]),
                             deq_pair<DT>(cA[3], sk[3], zk[3]), deq_pair<DT>(cB[3], sk[3], zk[3]), qk0[2 * k + 1], qk2[2 * k + 1]);
              }
              // this thread: tokens ra_ and ra_ + 8 of the page, query rows colp and colp + 1
              if (colp < rows) {
                float* scol = S + t * kUnit + warp * kQ4Page + ra_;
                const float g0 = gq[slot0 * kQ4Page + ra_], g8 = gq[slot0 * kQ4Page + ra_ + 8];
                const float s00 = (acc0[0] + acc1[0]) * (g0 * p.scale_log2), s08 = (acc0[2] + acc1[2]) * (g8 * p.scale_log2);
                if (!is_retained_scale(g0)) {
                  scol[colp * s_stride] = s00;
                  mx0 = fmaxf(mx0, s00);
                }
                if (!is_retained_scale(g8)) {
                  scol[colp * s_stride + 8] = s08;
                  mx0 = fmaxf(mx0, s08);
                }
                if (colp + 1 < rows) {
                  const float h0 = gq[slot1 * kQ4Page + ra_], h8 = gq[slot1 * kQ4Page + ra_ + 8];
                  const float s10 = (acc0[1] + acc1[1]) * (h0 * p.scale_log2), s18 = (acc0[3] + acc1[3]) * (h8 * p.scale_log2);
                  if (!is_retained_scale(h0)) {
                    scol[(colp + 1) * s_stride] = s10;
                    mx1 = fmaxf(mx1, s10);
                  }
                  if (!is_retained_scale(h8)) {
                    scol[(colp + 1) * s_stride + 8] = s18;
                    mx1 = fmaxf(mx1, s18);
                  }
                }
              }
            }
          }
          __syncwarp();
          if (lane == 0) mbar_arrive(empty0 + 8 * s);
          continue;
        }
        // a 16-bit tile stage: 64 tokens of pages, or (4-bit cache) the residual tile behind the 4-bit pages
        const int s_off = Q4 ? w.n_q : t * kTile;
        const int valid = Q4 ? w.n_tok - w.n_q : min(kTile, w.n_tok - t * kTile);
        if (Q4) load_qa();
        if (tk_w < valid) {
          // A = the warp's 16 token rows (k step: 16 channels), B = the query rows: D[token][row]
          float acc0[4] = {0.f, 0.f, 0.f, 0.f}, acc1[4] = {0.f, 0.f, 0.f, 0.f};  // even / odd k steps
          const int tk_m = tk_w + (mi & 1) * 8 + mr;  // token row this lane addresses for ldmatrix
          const uint32_t rowaddr = sbase + (uint32_t)((tk_m >> shift) * tbytes + (tk_m & (ps - 1)) * kRowBytes);
          // all eight loads first, then the contractions: the loads' latencies overlap
          uint32_t ra[8][4];
#pragma unroll
          for (int ks = 0; ks < 8; ++ks) {
            const int c = ks * 2 + (mi >> 1);
            ldsm_x4(rowaddr + ((uint32_t)((c & 8) | ((c & 7) ^ mr)) << 4), ra[ks][0], ra[ks][1], ra[ks][2], ra[ks][3]);
          }
#pragma unroll
          for (int ks = 0; ks < 8; ks += 2) {
            mma_rows<DT>(acc0, ra[ks][0], ra[ks][1], ra[ks][2], ra[ks][3], qa0[ks], qa2[ks]);
            mma_rows<DT>(acc1, ra[ks + 1][0], ra[ks + 1][1], ra[ks + 1][2], ra[ks + 1][3], qa0[ks + 1], qa2[ks + 1]);
          }
          // this thread: tokens tk_w + row and + 8, query rows colp and colp + 1.  A retained token
          // (scale = -0) gets its score from its raw row further down; past the last token nothing is stored.
          if (colp < rows) {
            const int tk = tk_w + row;
            const float* sc = reinterpret_cast<const float*>(stages + s * STAGE_BYTES + (tk >> shift) * tbytes + ps * kRowBytes) +
                              (tk & (ps - 1));
            const float* sc8 = reinterpret_cast<const float*>(stages + s * STAGE_BYTES + ((tk + 8) >> shift) * tbytes +
                                                              ps * kRowBytes) + ((tk + 8) & (ps - 1));
            float* scol = S + s_off + tk;
            const float g0 = sc[slot0 * ps], g8 = sc8[slot0 * ps];
            const bool u0 = tk < valid && !is_retained_scale(g0), u8 = tk + 8 < valid && !is_retained_scale(g8);
            const float s00 = (acc0[0] + acc1[0]) * (g0 * p.scale_log2), s08 = (acc0[2] + acc1[2]) * (g8 * p.scale_log2);
            if (u0) {
              scol[colp * s_stride] = s00;
              mx0 = fmaxf(mx0, s00);
            }
            if (u8) {
              scol[colp * s_stride + 8] = s08;
              mx0 = fmaxf(mx0, s08);
            }
            if (colp + 1 < rows) {
              const float h0 = sc[slot1 * ps], h8 = sc8[slot1 * ps];
              const float s10 = (acc0[1] + acc1[1]) * (h0 * p.scale_log2), s18 = (acc0[3] + acc1[3]) * (h8 * p.scale_log2);
              if (tk < valid && !is_retained_scale(h0)) {
                scol[(colp + 1) * s_stride] = s10;
                mx1 = fmaxf(mx1, s10);
              }
              if (tk + 8 < valid && !is_retained_scale(h8)) {
                scol[(colp + 1) * s_stride + 8] = s18;
                mx1 = fmaxf(mx1, s18);
              }
            }
          }
        }
        __syncwarp();
        if (lane == 0) mbar_arrive(empty0 + 8 * s);
      }
      // ---- retained K rows and the new token: their scores fill the columns the tiles left out.
      if (Q4 && xk > 0) load_qa();
      for (int x = 0; x < xk && ok; ++x, ++it) {
        const int s = it % N_STAGES;
        if (!mbar_wait(full0 + 8 * s, (it / N_STAGES) & 1, s_abort, p.status)) { ok = false; break; }
        const int cnt = info_s[2 * s];
        // single layer: warp w takes entries 8w..8w+7; pair mode: warps 0,1 layer l-1, warps 2,3 layer l
        const int set = nslots == 2 ? (warp >> 1) : 0;
        const int e_w = nslots == 2 ? (warp & 1) * 8 : warp * 8;
        if (e_w < cnt) {
          float acc0[4] = {0.f, 0.f, 0.f, 0.f};
          const unsigned char* sb = stages + s * STAGE_BYTES + set * set_bytes;
          const uint32_t rowaddr = smem_u32(sb) + (uint32_t)((e_w + mr) * kEntryBytes);
#pragma unroll
          for (int k2 = 0; k2 < 4; ++k2) {
            uint32_t r0, r1, r2, r3;  // (k step 2 k2: chunks lo, hi), (k step 2 k2 + 1: lo, hi)
            ldsm_x4(rowaddr + (uint32_t)((k2 * 4 + mi) << 4), r0, r1, r2, r3);
            mma_16816<DT>(acc0, qa0[2 * k2], qa2[2 * k2], r0, r1);
            mma_16816<DT>(acc0, qa0[2 * k2 + 1], qa2[2 * k2 + 1], r2, r3);
          }
          if (row < rows && set_row == set) {
#pragma unroll
            for (int k = 0; k < 2; ++k) {
              const int e = e_w + colp + k;
              if (e < cnt) {
                const int col = *reinterpret_cast<const int*>(sb + e * kEntryBytes + kRowBytes) - w.split_start;
                const float sc = acc0[k] * p.scale_log2;
                if (MC_IN_BOUNDS(col >= 0 && col <= w.n_tok, p.status)) {  // (the step's new token sits at column n_tok)
                  S[row * s_stride + col] = sc;
                  mxe = fmaxf(mxe, sc);
                }
              }
            }
          }
        }
        __syncwarp();
        if (lane == 0) mbar_arrive(empty0 + 8 * s);
      }
    }
    // ---- row maxima: every thread has tracked the scores it stored; the exponentials are taken
    // where the probabilities are used (V phase), so the scores are not passed over again ----------
#pragma unroll
    for (int o = 4; o < 32; o <<= 1) {
      mx0 = fmaxf(mx0, __shfl_xor_sync(0xffffffffu, mx0, o));
      mx1 = fmaxf(mx1, __shfl_xor_sync(0xffffffffu, mx1, o));
    }
    mxe = fmaxf(mxe, __shfl_xor_sync(0xffffffffu, mxe, 1));
    mxe = fmaxf(mxe, __shfl_xor_sync(0xffffffffu, mxe, 2));
    if (lane < 4) {
      red_s[colp * kConsumerWarps + warp] = mx0;        // rows colp, colp + 1 (tiles)
      red_s[(colp + 1) * kConsumerWarps + warp] = mx1;
    }
    if ((lane & 3) == 0) red2_s[row * kConsumerWarps + warp] = mxe;  // row `row` (raw rows)
    consumer_sync();
    auto row_max = [&](int r) {
      const float4 ma = *reinterpret_cast<const float4*>(red_s + r * kConsumerWarps);
      const float4 mb = *reinterpret_cast<const float4*>(red2_s + r * kConsumerWarps);
      return fmaxf(fmaxf(fmaxf(ma.x, ma.y), fmaxf(ma.z, ma.w)), fmaxf(fmaxf(mb.x, mb.y), fmaxf(mb.z, mb.w)));
    };
    // this chunk's maxima joined with the piece's so far; what was summed under the old maximum is
    // rescaled by 2^(old - new)
    auto rescale = [](float m_old, float m_new) { return m_old == -INFINITY ? 0.f : exp2f(m_old - m_new); };
    if (w.first) {
      m_run = m_run0 = m_run1 = -INFINITY;
      l_acc = 0.f;
#pragma unroll
      for (int a = 0; a < 8; ++a)
#pragma unroll
        for (int k = 0; k < 4; ++k) acc[a][k] = 0.f;
    }
    const float m_row = fmaxf(m_run, row_max(row));
    if (!w.first) {
      const float m0 = fmaxf(m_run0, row_max(colp)), m1 = fmaxf(m_run1, row_max(colp + 1));
      const float f = rescale(m_run, m_row), f0 = rescale(m_run0, m0), f1 = rescale(m_run1, m1);
      l_acc *= f;
#pragma unroll
      for (int a = 0; a < 8; ++a) {
        acc[a][0] *= f0;
        acc[a][2] *= f0;
        acc[a][1] *= f1;
        acc[a][3] *= f1;
      }
      m_run0 = m0;
      m_run1 = m1;
    } else {
      m_run0 = row_max(colp);
      m_run1 = row_max(colp + 1);
    }
    m_run = m_row;
    if (w.last && warp == 0 && (lane & 3) == 0) m_s[row] = m_row;

    // query rows of the next item travel while the V tiles stream
    uint32_t qnext[4];
    load_q_words(piece_at<Q4>(cur, x_begin, x_end, pre_s, len_s, p), qnext);

    // ---- V phase: O[r][:] = sum_i (P[r][i] g_i) e_i -----------------------------------------------
    // A = the warp's 16 token rows transposed (16 channels x 16 tokens per m tile), B = the rows'
    // probabilities times the V scale: D[channel][row], eight m tiles = all 128 channels.  Every
    // warp sums its own tokens; the four partial sums meet in shared memory after the piece's last chunk.
    const int tk_w = warp * 16;
    // chunk position of m tile j for this lane: chunk 2 j + (mi & 1) of a row whose index is mr (mod 8)
    const uint32_t vsw_lo = (uint32_t)(((mi & 1) ^ (mr & 1)) | (mr & 6));
    if (ok) {
      int xv = n_new;
      for (int t = 0; t < w.TT; ++t, ++it) {
        const int s = it % N_STAGES;
        if (!mbar_wait(full0 + 8 * s, (it / N_STAGES) & 1, s_abort, p.status)) { ok = false; break; }
        const uint32_t sbase = stage0 + s * STAGE_BYTES;
        xv = info_s[2 * s + 1];
        if (Q4 && t < w.Tq) {
          // ---- four 4-bit pages, one per warp: lane (row, t4) owns the channels row, row + 8 (mod 16)
          // of the token pairs t4, t4 + 4 of each half page: one 16-byte chunk of codes per pair
          if (warp < (w.n_q >> 5) - t * (kUnit / kQ4Page)) {
            const unsigned char* tb = stages + s * STAGE_BYTES + warp * kQ4TileBytes;
            const int t4 = lane & 3;
            const float* gq = reinterpret_cast<const float*>(tb + kQ4ScaleOff) + slot_row * kQ4Page;
            const float* srow = S + row * s_stride + t * kUnit + warp * kQ4Page;
#pragma unroll
            for (int hf = 0; hf < 2; ++hf) {
              // B fragment: row `row`, tokens 16 hf + colp, + 1, + 8, + 9 of the page
              uint32_t b0 = 0u, b1 = 0u;
              if (row < rows) {
                const float2 p0 = *reinterpret_cast<const float2*>(srow + 16 * hf + colp);
                const float2 p1 = *reinterpret_cast<const float2*>(srow + 16 * hf + 8 + colp);
                const float2 g0 = *reinterpret_cast<const float2*>(gq + 16 * hf + colp);
                const float2 g1 = *reinterpret_cast<const float2*>(gq + 16 * hf + 8 + colp);
                // (a retained token's column holds the score of its raw row; its scale -0 removes it here)
                const float e0 = exp2f(p0.x - m_row), e1 = exp2f(p0.y - m_row);
                const float e2 = exp2f(p1.x - m_row), e3 = exp2f(p1.y - m_row);
                l_acc += (e0 + e1) + (e2 + e3);
                b0 = Elem<DT>::pack(e0 * g0.x, e1 * g0.y);
                b1 = Elem<DT>::pack(e2 * g1.x, e3 * g1.y);
              }
              const int i0 = 8 * hf + t4, i1 = i0 + 4;  // token pairs (2 i0, 2 i0 + 1), (2 i1, 2 i1 + 1)
              const uint32_t cpos = (uint32_t)(row ^ (t4 << 1)) << 4;
              const uint4 w0 = *reinterpret_cast<const uint4*>(tb + i0 * 128 + cpos);
              const uint4 w1 = *reinterpret_cast<const uint4*>(tb + i1 * 128 + cpos);
              const uint4 s0 = *reinterpret_cast<const uint4*>(tb + kQ4CodeBytes + i0 * 32);
              const uint4 z0 = *reinterpret_cast<const uint4*>(tb + kQ4CodeBytes + i0 * 32 + 16);
              const uint4 s1 = *reinterpret_cast<const uint4*>(tb + kQ4CodeBytes + i1 * 32);
              const uint4 z1 = *reinterpret_cast<const uint4*>(tb + kQ4CodeBytes + i1 * 32 + 16);
              const uint32_t w0a[4] = {w0.x, w0.y, w0.z, w0.w}, w1a[4] = {w1.x, w1.y, w1.z, w1.w};
              const uint32_t s0a[4] = {s0.x, s0.y, s0.z, s0.w}, z0a[4] = {z0.x, z0.y, z0.z, z0.w};
              const uint32_t s1a[4] = {s1.x, s1.y, s1.z, s1.w}, z1a[4] = {z1.x, z1.y, z1.z, z1.w};
#pragma unroll
              for (int k = 0; k < 4; ++k) {  // word k = channel group k: m tiles 2 k and 2 k + 1
                uint32_t c0[4], c1[4];
                code_pairs<DT>(w0a[k], c0);
                code_pairs<DT>(w1a[k], c1);
                mma_rows<DT>(acc[2 * k], deq_pair<DT>(c0[0], s0a[k], z0a[k]), deq_pair<DT>(c0[1], s0a[k], z0a[k]),
                             deq_pair<DT>(c1[0], s1a[k], z1a[k]), deq_pair<DT>(c1[1], s1a[k], z1a[k]), b0, b1);
                mma_rows<DT>(acc[2 * k + 1], deq_pair<DT>(c0[2], s0a[k], z0a[k]), deq_pair<DT>(c0[3], s0a[k], z0a[k]),
                             deq_pair<DT>(c1[2], s1a[k], z1a[k]), deq_pair<DT>(c1[3], s1a[k], z1a[k]), b0, b1);
              }
            }
          }
          __syncwarp();
          if (lane == 0) mbar_arrive(empty0 + 8 * s);
          continue;
        }
        const int s_off = Q4 ? w.n_q : t * kTile;
        const int valid = Q4 ? w.n_tok - w.n_q : min(kTile, w.n_tok - t * kTile);
        bool wrote = false;
        if (tk_w < valid) {
          if (valid < tk_w + 16) {
            // rows past the last cached token may hold anything (page tail, page not copied): zero
            // them so that 0 * x stays 0 in the contraction
            for (int i = lane; i < (tk_w + 16 - valid) * 16; i += 32) {
              const uint32_t a = tile_addr(sbase, valid + (i >> 4), i & 15, shift, tbytes);
              asm volatile("st.shared.v4.u32 [%0], {%1,%1,%1,%1};" ::"r"(a), "r"(0u) : "memory");
            }
            wrote = true;
            __syncwarp();
          }
          // B fragment: row `row`, tokens tk_w + colp, + 1, + 8, + 9
          uint32_t b0 = 0u, b1 = 0u;
          if (row < rows) {
            const float* scj = reinterpret_cast<const float*>(stages + s * STAGE_BYTES + (tk_w >> shift) * tbytes +
                                                              ps * kRowBytes) + slot_row * ps + (tk_w & (ps - 1));
            const float* srow = S + row * s_stride + s_off + tk_w;
            const float2 p0 = *reinterpret_cast<const float2*>(srow + colp);
            const float2 p1 = *reinterpret_cast<const float2*>(srow + 8 + colp);
            const float2 g0 = *reinterpret_cast<const float2*>(scj + colp);
            const float2 g1 = *reinterpret_cast<const float2*>(scj + 8 + colp);
            const int c0 = tk_w + colp;
            const float e0 = c0 < valid ? exp2f(p0.x - m_row) : 0.f, e1 = c0 + 1 < valid ? exp2f(p0.y - m_row) : 0.f;
            const float e2 = c0 + 8 < valid ? exp2f(p1.x - m_row) : 0.f, e3 = c0 + 9 < valid ? exp2f(p1.y - m_row) : 0.f;
            l_acc += (e0 + e1) + (e2 + e3);
            b0 = Elem<DT>::pack(e0 * g0.x, e1 * g0.y);
            b1 = Elem<DT>::pack(e2 * g1.x, e3 * g1.y);
          }
          const int tk_m = tk_w + (mi >> 1) * 8 + mr;  // token row this lane addresses for ldmatrix
          const uint32_t rowaddr = sbase + (uint32_t)((tk_m >> shift) * tbytes + (tk_m & (ps - 1)) * kRowBytes);
          uint32_t ra[8][4];  // all eight loads first, then the contractions
#pragma unroll
          for (int j = 0; j < 8; ++j)
            ldsm_x4_t(rowaddr + (((uint32_t)((j >> 2) << 3) | ((uint32_t)(2 * (j & 3)) ^ vsw_lo)) << 4), ra[j][0], ra[j][1],
                      ra[j][2], ra[j][3]);
#pragma unroll
          for (int j = 0; j < 8; ++j) mma_rows<DT>(acc[j], ra[j][0], ra[j][1], ra[j][2], ra[j][3], b0, b1);
        }
        if (__any_sync(0xffffffffu, wrote)) asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
        __syncwarp();
        if (lane == 0) mbar_arrive(empty0 + 8 * s);
      }
      // ---- retained V rows and the new token: raw rows weighted by their tokens' probabilities.
      // Single layer: warp w takes entries 16 w .. 16 w + 15; pair mode (16 entries per layer):
      // warp 0 layer l-1, warp 2 layer l.
      for (int x = 0; x < xv && ok; ++x, ++it) {
        const int s = it % N_STAGES;
        if (!mbar_wait(full0 + 8 * s, (it / N_STAGES) & 1, s_abort, p.status)) { ok = false; break; }
        const int cnt = info_s[2 * s];
        const int set = nslots == 2 ? (warp >> 1) : 0;
        const int e_w = nslots == 2 ? (warp & 1) * 16 : warp * 16;
        bool wrote = false;
        if (e_w < cnt) {
          const unsigned char* sb = stages + s * STAGE_BYTES + set * set_bytes;
          const uint32_t sba = smem_u32(sb);
          if (cnt < e_w + 16) {  // entries past the last one: zero
            for (int i = lane; i < (e_w + 16 - cnt) * 16; i += 32) {
              const uint32_t a = sba + (uint32_t)((cnt + (i >> 4)) * kEntryBytes + ((i & 15) << 4));
              asm volatile("st.shared.v4.u32 [%0], {%1,%1,%1,%1};" ::"r"(a), "r"(0u) : "memory");
            }
            wrote = true;
            __syncwarp();
          }
          uint32_t b0 = 0u, b1 = 0u;
          if (row < rows && set_row == set) {
            float pv[4];
#pragma unroll
            for (int k = 0; k < 4; ++k) {
              const int e = e_w + colp + (k & 1) + (k >> 1) * 8;
              pv[k] = 0.f;
              if (e < cnt) {
                const int col = *reinterpret_cast<const int*>(sb + e * kEntryBytes + kRowBytes) - w.split_start;
                if (MC_IN_BOUNDS(col >= 0 && col <= w.n_tok, p.status)) {
                  pv[k] = exp2f(S[row * s_stride + col] - m_row);
                  if (col >= w.n_tok) l_acc += pv[k];  // the new token: no tile has counted it
                }
              }
            }
            b0 = Elem<DT>::pack(pv[0], pv[1]);
            b1 = Elem<DT>::pack(pv[2], pv[3]);
          }
          const uint32_t rowaddr = sba + (uint32_t)((e_w + (mi >> 1) * 8 + mr) * kEntryBytes + ((mi & 1) << 4));
#pragma unroll
          for (int j = 0; j < 8; ++j) {
            uint32_t a0, a1, a2, a3;
            ldsm_x4_t(rowaddr + (uint32_t)(j << 5), a0, a1, a2, a3);
            mma_rows<DT>(acc[j], a0, a1, a2, a3, b0, b1);
          }
        }
        if (__any_sync(0xffffffffu, wrote)) asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
        __syncwarp();
        if (lane == 0) mbar_arrive(empty0 + 8 * s);
      }
    }

    // ---- the piece's partial result after its last chunk: the four warps' sums meet in shared
    // memory (the score buffer, free once every warp has left the V phase) ----------------------------
    if (w.last) {
    l_acc += __shfl_xor_sync(0xffffffffu, l_acc, 1);
    l_acc += __shfl_xor_sync(0xffffffffu, l_acc, 2);
    if ((lane & 3) == 0) l_s[row * kConsumerWarps + warp] = l_acc;
    consumer_sync();
    {
      float* slab = S + warp * rows * kSlabStride;  // [rows][kSlabStride]
#pragma unroll
      for (int j = 0; j < 8; ++j) {
        const int ch = j * 16 + row;
        if (colp < rows) {
          slab[colp * kSlabStride + ch] = acc[j][0];
          slab[colp * kSlabStride + ch + 8] = acc[j][2];
        }
        if (colp + 1 < rows) {
          slab[(colp + 1) * kSlabStride + ch] = acc[j][1];
          slab[(colp + 1) * kSlabStride + ch + 8] = acc[j][3];
        }
      }
    }
    consumer_sync();
    for (int r = 0; r < rows; ++r) {
      const int set_r = nslots == 2 ? r / p.nq : 0;
      const int rq = r - set_r * p.nq;
      const size_t prow = (((size_t)set_r * p.g.batch + w.b) * p.n_q_heads + w.g * p.nq + rq) * p.slots + w.split;
      const float* sl = S + r * kSlabStride + tid;
      const int ws = rows * kSlabStride;
      p.part_o[prow * kHeadDim + tid] = (sl[0] + sl[ws]) + (sl[2 * ws] + sl[3 * ws]);
      if (tid == 0) {
        const float4 ll = *reinterpret_cast<const float4*>(l_s + r * kConsumerWarps);
        p.part_ml[prow * 2] = m_s[r];
        p.part_ml[prow * 2 + 1] = (ll.x + ll.y) + (ll.z + ll.w);
      }
    }
    }
    // next item's query rows into the other buffer (nobody reads that buffer any more)
    {
      uint32_t* qn = q_s + ((n_item + 1) & 1) * kMaxRows * 64;
#pragma unroll
      for (int k = 0; k < 4; ++k) qn[tid + k * kConsumerThreads] = qnext[k];
    }
    consumer_sync();
    if (*s_abort) break;  // read after the barrier: the same answer in every consumer thread
  }
  if (*s_abort) {
    // give copies that may still be in flight time to land before the CTA's memory is released
    for (int k = 0; k < 2000; ++k) __nanosleep(1000);
  }
}

// Log-sum-exp merge of the pieces' partials: out = sum_j 2^(m_j - M) o_j / sum_j 2^(m_j - M) l_j.
// A block serves R query heads of one sequence (R = 8: a warp per output row, for batches with many
// rows; R = 1: the eight warps share the pieces of one row, for few rows with many pieces); a lane
// owns four channels.  The pieces of the sequence follow from the lengths and the number of teams: one per
// team range that touches the sequence, stored in the slot of its first unit; a thread per such team
// writes the list into shared memory, before the wait on the split kernel (the lengths belong to the
// caller), whose tail this overlaps.
constexpr int kCombineThreads = 256;
constexpr int kCombineWarps = kCombineThreads / 32;
constexpr int kMaxPieces = 2048;  // pieces of one sequence = teams (checked on the host)

// The launch can carry the decode step's append as well (mc_decode_attn_append): blocks past the combine's own
// (blockIdx.x >= combine_x) merge the new token pair of sequence blockIdx.y into the pair cache, a row per
// half-warp -- what append_kernel does, without a launch of its own.  The split kernel is complete by then
// (the wait), so nothing reads the cache while the row is written.
template <int DT, int R>
__global__ void __launch_bounds__(kCombineThreads) attn_combine_kernel(const AttnParams p, unsigned short* out, float* lse,
                                                                       const __grid_constant__ AppendParams app, int combine_x) {
  grid_dep_launch();
  if ((int)blockIdx.x >= combine_x) {
    const int H = app.g.n_kv_heads;
    const int j = ((int)blockIdx.x - combine_x) * (kCombineThreads / 16) + (int)(threadIdx.x >> 4);  // (tensor, head) of the sequence
    const int r = blockIdx.z == 0 && j < 2 * H ? ((j / H) * app.g.batch + (int)blockIdx.y) * H + j % H : app.total_rows;
    append_row<DT>(app, r, threadIdx.x & 15, [] { grid_dep_wait(); });
    return;
  }
  constexpr int GP = kCombineWarps / R;  // warps per output row
  __shared__ int sum_s[2][kCombineWarps];
  __shared__ int list_s[kMaxPieces];
  __shared__ float red_s[kCombineWarps];
  __shared__ float4 acc_s[GP > 1 ? kCombineWarps : 1][32];
  const int b = blockIdx.y, set = blockIdx.z;
  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  const int grp = warp % GP;  // this warp takes the pieces grp, grp + GP, ... of its row
  const int hq = blockIdx.x * R + warp / GP;
  int before = 0, all = 0;  // units of the sequences before this one, of all sequences
  for (int bb = tid; bb < p.g.batch; bb += kCombineThreads) {
    const int ub = max(1, (min(max(p.g.seq_lens[bb], 0), p.g.max_seq_len) + kUnit - 1) / kUnit);
    all += ub;
    if (bb < b) before += ub;
  }
  for (int o = 16; o; o >>= 1) {
    before += __shfl_xor_sync(0xffffffffu, before, o);
    all += __shfl_xor_sync(0xffffffffu, all, o);
  }
  if (lane == 0) {
    sum_s[0][warp] = before;
    sum_s[1][warp] = all;
  }
  __syncthreads();
  before = 0;
  all = 0;
#pragma unroll
  for (int g = 0; g < kCombineWarps; ++g) {
    before += sum_s[0][g];
    all += sum_s[1][g];
  }
  const int u = max(1, (min(max(p.g.seq_lens[b], 0), p.g.max_seq_len) + kUnit - 1) / kUnit);
  const long long n_units = all, x0 = before;
  const int n_teams = p.n_teams;
  // teams whose range [n_units c / T, n_units (c + 1) / T) meets [x0, x0 + u): consecutive, each with one piece
  const int c_first = (int)(((x0 + 1) * n_teams - 1) / n_units);
  const int c_last = (int)(((x0 + u) * n_teams - 1) / n_units);
  // (a team's range can be empty when there are fewer units than teams: count, scan, then write)
  int base = 0;
  for (int c0 = c_first; c0 <= c_last; c0 += kCombineThreads) {  // (more teams than threads: one more round)
    const int c = c0 + tid;
    int s0 = 0, cnt = 0;
    if (c <= c_last) {
      const long long lo = max(x0, n_units * c / n_teams), hi = min(x0 + u, n_units * (c + 1) / n_teams);
      s0 = (int)(lo - x0);
      cnt = hi > lo ? 1 : 0;
    }
    int incl = cnt;
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) {
      const int v = __shfl_up_sync(0xffffffffu, incl, o);
      if (lane >= o) incl += v;
    }
    __syncthreads();  // sum_s is free again
    if (lane == 31) sum_s[0][warp] = incl;
    __syncthreads();
    int off = base + incl - cnt;
    for (int g = 0; g < warp; ++g) off += sum_s[0][g];
    if (cnt && off < kMaxPieces) list_s[off] = s0;
#pragma unroll
    for (int g = 0; g < kCombineWarps; ++g) base += sum_s[0][g];
  }
  const int n = min(base, kMaxPieces);
  __syncthreads();
  grid_dep_wait();
  const bool active = hq < p.n_q_heads;
  if (GP == 1 && !active) return;
  const size_t prow0 = (((size_t)set * p.g.batch + b) * p.n_q_heads + hq) * p.slots;
  const float2* ml = reinterpret_cast<const float2*>(p.part_ml) + prow0;
  const float4* po = reinterpret_cast<const float4*>(p.part_o + prow0 * kHeadDim) + lane;
  // The first four pieces are requested before anything depends on a loaded value, so the maxima
  // and these partials arrive together.
  float2 v2[4];
  float4 v[4];
  auto load4 = [&](int j0) {
#pragma unroll
    for (int k = 0; k < 4; ++k) {
      v2[k] = make_float2(-INFINITY, 0.f);
      v[k] = make_float4(0.f, 0.f, 0.f, 0.f);
      if (active && j0 + k * GP < n) {
        const int slot = list_s[j0 + k * GP];
        v2[k] = ml[slot];
        v[k] = po[(size_t)slot * (kHeadDim / 4)];
      }
    }
  };
  load4(grp);
  float M = -INFINITY;
  if (active)
    for (int j = lane; j < n; j += 32) M = fmaxf(M, ml[list_s[j]].x);
  for (int o = 16; o; o >>= 1) M = fmaxf(M, __shfl_xor_sync(0xffffffffu, M, o));
  float L = 0.f;
  float4 o = make_float4(0.f, 0.f, 0.f, 0.f);
  for (int j0 = grp; j0 < n; j0 += 4 * GP) {
    if (j0 != grp) load4(j0);
#pragma unroll
    for (int k = 0; k < 4; ++k) {
      const float w = v2[k].x == -INFINITY ? 0.f : exp2f(v2[k].x - M);
      L = fmaf(w, v2[k].y, L);
      o.x = fmaf(w, v[k].x, o.x);
      o.y = fmaf(w, v[k].y, o.y);
      o.z = fmaf(w, v[k].z, o.z);
      o.w = fmaf(w, v[k].w, o.w);
    }
  }
  if (GP > 1) {  // the row's warps meet in shared memory
    acc_s[GP > 1 ? warp : 0][lane] = o;
    if (lane == 0) red_s[warp] = L;
    __syncthreads();
    if (grp != 0 || !active) return;
    for (int g = 1; g < GP; ++g) {
      const float4 t = acc_s[GP > 1 ? warp + g : 0][lane];
      L += red_s[warp + g];
      o.x += t.x;
      o.y += t.y;
      o.z += t.z;
      o.w += t.w;
    }
  }
  const float inv = L > 0.f ? 1.f / L : 0.f;
  const size_t orow = ((size_t)set * p.g.batch + b) * p.n_q_heads + hq;
  uint2 packed;
  packed.x = Elem<DT>::pack(o.x * inv, o.y * inv);
  packed.y = Elem<DT>::pack(o.z * inv, o.w * inv);
  *reinterpret_cast<uint2*>(out + orow * kHeadDim + lane * 4) = packed;
  if (lse != nullptr && lane == 0) lse[orow] = L > 0.f ? (M + log2f(L)) * 0.69314718055994530942f : -INFINITY;
}

// ---- host side ------------------------------------------------------------------------------------
static size_t attn_smem_bytes(bool q4, bool wide) {
  size_t b = 128 + (q4 ? (size_t)kQ4Stages * kQ4StageBytes : (size_t)(wide ? kStagesWide : kStages) * kStageBytes) +
             (size_t)(wide ? kScoreFloatsWide : kScoreFloats) * 4;  // stages, S
  b += 2 * kMaxRows * 64 * 4;                                                  // q_s
  b += kMaxRows * 4 + 3 * kMaxRows * kConsumerWarps * 4;                       // m, l, red, red2
  b += 2 * kStages * 4 + (2 * kMaxBatchSmem + 1) * 4 + 2 * kMaxPiecePages * 4 + 4 + 8 + 2 * kStages * 8 + 64;
  return b;
}

// Partial slots per output row: the units of the longest sequence.
static size_t attn_slots(const mc_batch* bt) { return (size_t)std::max(1, (bt->max_seq_len + kUnit - 1) / kUnit); }

size_t attn_workspace_bytes(const mc_config* cfg, const mc_batch* bt, int n_sets) {
  const size_t prow = (size_t)n_sets * bt->batch * cfg->n_q_heads * attn_slots(bt);
  return align_up(prow * kHeadDim * 4, 256) + align_up(prow * 2 * 4, 256);
}

mc_status launch_decode_attn(const mc_config* cfg, const mc_batch* bt, const Geom& g, const mc_pair_cache* pair,
                             int layer_sel, const void* q, const void* k_new, const void* v_new, float sm_scale,
                             void* out, float* lse, void* workspace, cudaStream_t stream, const AppendParams* append) {
  if (bt->batch == 0) return MC_OK;
  if (bt->batch > kMaxBatchSmem) return MC_ERR_SHAPE;
  AttnParams ap;
  ap.g = g;
  ap.e_pool[0] = (const char*)pair->e_k;
  ap.e_pool[1] = (const char*)pair->e_v;
  const bool q4 = cfg->cache_bits == 4;
  ap.res_pool[0] = q4 ? (const char*)pair->res_k : nullptr;
  ap.res_pool[1] = q4 ? (const char*)pair->res_v : nullptr;
  ap.ret_offset = pair->ret_offset;
  ap.ret_prefix = pair->ret_prefix;
  ap.ret_prefix_stride = (int)pair->ret_prefix_stride;
  ap.ret_rows = (const char*)pair->ret_rows;
  ap.ret_capacity = pair->ret_capacity;
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
  const bool wide = q4 || ap.rows > 1;  // (see kScoreFloatsWide)
  ap.cap_units = piece_cap_units(ap.rows, wide);
  ap.slots = (int)attn_slots(bt);
  const size_t prow = (size_t)ap.n_sets * bt->batch * cfg->n_q_heads * ap.slots;
  ap.part_o = reinterpret_cast<float*>(workspace);
  ap.part_ml = reinterpret_cast<float*>((char*)workspace + align_up(prow * kHeadDim * 4, 256));

  int n_sm = 0;  // persistent grid: kCtasPerSm CTAs per SM of the current device
  if (mc_status st = sm_count(&n_sm)) return st;
  // teams: S CTAs, each with ceil(H / S) kv heads; as many whole teams as fit two CTAs per SM,
  // and no more teams than there can be units
  const int slots_gpu = n_sm * kCtasPerSm;
  const int heads_per_cta = (cfg->n_kv_heads + std::min(slots_gpu, 32) - 1) / std::min(slots_gpu, 32);
  ap.team_size = (cfg->n_kv_heads + heads_per_cta - 1) / heads_per_cta;
  const long long max_units = (long long)bt->batch * ap.slots;
  const int n_teams = (int)std::max<long long>(1, std::min<long long>(slots_gpu / ap.team_size, max_units));
  const int grid = n_teams * ap.team_size;
  ap.n_teams = n_teams;
  if (n_teams > kMaxPieces) return MC_ERR_SHAPE;  // pieces of one sequence
  const size_t smem = attn_smem_bytes(q4, wide);
  // many output rows: a warp per row; few: a block per row
  const bool warp_rows = (long long)ap.n_sets * bt->batch * cfg->n_q_heads >= 1024;
  dim3 cgrid(warp_rows ? (cfg->n_q_heads + kCombineWarps - 1) / kCombineWarps : cfg->n_q_heads, bt->batch, ap.n_sets);
  void (*split)(const AttnParams) =
      cfg->dtype == MC_F16
          ? (q4 ? attn_split_kernel<MC_F16, true, true> : (wide ? attn_split_kernel<MC_F16, false, true> : attn_split_kernel<MC_F16, false, false>))
          : (q4 ? attn_split_kernel<MC_BF16, true, true> : (wide ? attn_split_kernel<MC_BF16, false, true> : attn_split_kernel<MC_BF16, false, false>));
  // (the append rides on the combine launch: ceil(2 H / 16) more blocks per sequence)
  AppendParams app;
  memset(&app, 0, sizeof(app));
  const int combine_x = (int)cgrid.x;
  if (append != nullptr) {
    app = *append;
    cgrid.x += (2 * cfg->n_kv_heads + kCombineThreads / 16 - 1) / (kCombineThreads / 16);
  }
  void (*combine)(const AttnParams, unsigned short*, float*, const AppendParams, int) =
      cfg->dtype == MC_F16 ? (warp_rows ? attn_combine_kernel<MC_F16, kCombineWarps> : attn_combine_kernel<MC_F16, 1>)
                           : (warp_rows ? attn_combine_kernel<MC_BF16, kCombineWarps> : attn_combine_kernel<MC_BF16, 1>);
  MC_CUDA_CHECK(cudaFuncSetAttribute(split, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem));
  MC_CUDA_CHECK(launch_pdl(split, dim3(grid), dim3(kAttnThreads), smem, stream, ap));
  MC_CUDA_CHECK(cudaGetLastError());
  MC_CUDA_CHECK(launch_pdl(combine, dim3(cgrid), dim3(kCombineThreads), 0, stream, ap, (unsigned short*)out, lse, app, combine_x));
  MC_CUDA_CHECK(cudaGetLastError());
  return MC_OK;
}

// ---- self-test of the bounded wait -------------------------------------------------------------------
// One warp waits on a barrier that nothing ever completes, with the wait the streaming kernels use
// (a short poll limit): the wait gives up, records MC_FLAG_WAIT_TIMEOUT in the status words and the
// kernel returns normally.
__global__ void __launch_bounds__(32) wait_timeout_probe_kernel(int32_t* status, uint32_t limit) {
  grid_dep_wait();
  grid_dep_launch();
  __shared__ uint64_t bar;
  __shared__ int s_abort;
  if (threadIdx.x == 0) {
    mbar_init(smem_u32(&bar), 1);
    s_abort = 0;
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  __syncwarp();
  if (threadIdx.x == 0) mbar_wait(smem_u32(&bar), 0, &s_abort, status, limit);
  __syncwarp();
}

mc_status launch_wait_timeout_probe(int32_t* status, uint32_t limit, cudaStream_t stream) {
  MC_CUDA_CHECK(launch_pdl(wait_timeout_probe_kernel, dim3(1), dim3(32), 0, stream, status, limit));
  MC_CUDA_CHECK(cudaGetLastError());
  return MC_OK;
}

// ---- new-token rows from device-addressable host memory ------------------------------------------
__global__ void __launch_bounds__(256) fetch_rows_kernel(const uint4* k_src, const uint4* v_src, uint4* k_dst, uint4* v_dst,
                                                         int n16) {
  grid_dep_launch();
  const int i = blockIdx.x * blockDim.x + threadIdx.x;
  uint4 a = make_uint4(0u, 0u, 0u, 0u), b = a;
  if (i < n16) {  // the caller's rows are read before the wait, the staging buffer written after it
    a = k_src[i];
    b = v_src[i];
  }
  grid_dep_wait();
  if (i < n16) {
    k_dst[i] = a;
    v_dst[i] = b;
  }
}

mc_status launch_fetch_rows(const void* k_src, const void* v_src, void* k_dst, void* v_dst, size_t n, cudaStream_t stream) {
  const int n16 = (int)(n / 16);
  if (n16 == 0) return MC_OK;
  MC_CUDA_CHECK(launch_pdl(fetch_rows_kernel, dim3((n16 + 255) / 256), dim3(256), 0, stream, (const uint4*)k_src,
                           (const uint4*)v_src, (uint4*)k_dst, (uint4*)v_dst, n16));
  MC_CUDA_CHECK(cudaGetLastError());
  return MC_OK;
}

// Up to three arrays (16-byte pieces) from device-addressable host memory into device memory, one launch.
struct Fetch3 {
  const uint4* src[3];
  uint4* dst[3];
  int n16[3];
};
__global__ void __launch_bounds__(256) fetch3_kernel(const Fetch3 f) {
  grid_dep_launch();
  const int a = blockIdx.y;
  const int i = blockIdx.x * blockDim.x + threadIdx.x;
  uint4 v = make_uint4(0u, 0u, 0u, 0u);
  if (i < f.n16[a]) v = f.src[a][i];  // the caller's rows are read before the wait, the staging buffer written after it
  grid_dep_wait();
  if (i < f.n16[a]) f.dst[a][i] = v;
}

mc_status launch_fetch3(const void* const* src, void* const* dst, const size_t* bytes, int n, cudaStream_t stream) {
  Fetch3 f;
  int most = 0;
  for (int a = 0; a < 3; ++a) {
    f.src[a] = a < n ? (const uint4*)src[a] : nullptr;
    f.dst[a] = a < n ? (uint4*)dst[a] : nullptr;
    f.n16[a] = a < n ? (int)(bytes[a] / 16) : 0;
    most = std::max(most, f.n16[a]);
  }
  if (most == 0) return MC_OK;
  MC_CUDA_CHECK(launch_pdl(fetch3_kernel, dim3((most + 255) / 256, n), dim3(256), 0, stream, f));
  MC_CUDA_CHECK(cudaGetLastError());
  return MC_OK;
}

}  // namespace mc

// ---------------------------------------------------------------------------------------------------
// Decode attention for callers that cannot supply scratch memory: the pieces' partials live in a
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
