/*
 * minicache.h -- C ABI of the MiniCache hot path for NVIDIA B200 (sm_100a).
 *
 * MiniCache (arXiv 2405.14366) compresses the KV cache in the depth dimension:
 * for every adjacent layer pair (l-1, l) from the start layer S = L/2 upwards
 * (Sec. 4.1), each key and value vector of both layers is split into magnitude
 * and unit direction (Eq. 2), the two directions are merged by spherical
 * interpolation with parameter t (Eq. 3), both magnitudes are kept, and the
 * token pairs whose angular distance d = Omega / pi stands out are kept
 * unmerged (Eq. 4).  At decode time a layer's K/V is the shared direction
 * times that layer's magnitude with the retained rows put back (Sec. 4.2
 * "Cache restoration"; Algorithm 2 "MiniCache Decoding").
 *
 * One "vector" here is one (token, kv head) row of 128 channels.  d_min and
 * d_max of Eq. 4 are taken per segment = (tensor K or V, sequence, kv head).
 *
 * General conventions
 * -------------------
 * - The device that is current when a call is made must be the one that owns `stream` and the
 *   buffers.
 * - Every pointer inside the structs below is DEVICE memory owned by the caller
 *   unless a comment says "host".  The library never allocates or frees device
 *   memory.  Struct arguments themselves live in host memory and are read
 *   before the call returns.
 * - All compute calls only enqueue work on `stream` (a cudaStream_t passed as
 *   void*, NULL = default stream) and return; they never synchronise.
 * - Pools are paged: [n_pages][n_kv_heads][page_size][128] elements of the
 *   16-bit storage type, base addresses 256-byte aligned.  One block table
 *   ([batch][max_pages_per_seq], int32 page ids) addresses every pool of a
 *   batch: page id p names slot p of the layer pools and of the pair cache
 *   alike.  Token i of sequence b lives in page block_table[b][i / page_size]
 *   at row i % page_size.
 * - The kernels are chained with programmatic dependent launch.  The batch description
 *   (block_table, seq_lens) and the queries are never written by this library, so
 *   mc_decode_attn and mc_append_pair read them before they wait for the kernel ahead in the stream; a
 *   caller whose own kernels let dependents start early must have them written before that.
 * - Argument errors are reported synchronously through the return code and
 *   launch nothing.  Data-dependent conditions (retained-row pool too small,
 *   a bounded wait inside a kernel running out) are recorded in the pair
 *   cache's device status words and read back with mc_read_status.
 * - Results are deterministic: identical inputs give bit-identical outputs.
 */
#ifndef MINICACHE_H_
#define MINICACHE_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef enum {
  MC_OK = 0,
  MC_ERR_INVALID_ARG = 1, /* null pointer, negative size, bad enum value */
  MC_ERR_SHAPE = 2,       /* head_dim != 128, page_size not 16/32/64, head ratio not supported,
                             batch above 1024 (merge, restore) or 512 (decode attention), or more than
                             65535 segments (2 * batch * n_kv_heads) */
  MC_ERR_DTYPE = 3,
  MC_ERR_ALIGN = 4,       /* a pool base is not 256-byte aligned */
  MC_ERR_CAPACITY = 5,    /* workspace too small / retained pool overflowed (from mc_read_status) */
  MC_ERR_UNSUPPORTED = 6,
  MC_ERR_CUDA = 7,        /* a CUDA runtime/driver call failed; see mc_last_cuda_error */
  MC_ERR_DEVICE_STATUS = 8 /* a kernel recorded a failure in the status words */
} mc_status;

typedef enum { MC_F16 = 0, MC_BF16 = 1 } mc_dtype;

/* Which tokens Eq. 4 keeps unmerged.
 * DISTINCT: d_i > d_max - (d_max - d_min) * gamma  (Eq. 4 applied to similarity 1 - d: the most
 *           distinct pairs are kept, as the text around Eq. 4 describes; gamma = 0 keeps none).
 * LITERAL : d_i < d_min + (d_max - d_min) * gamma  (Eq. 4 exactly as printed).
 * TOPK    : the ceil(gamma * n) largest d of the segment (ties: lower index first). */
typedef enum { MC_RETAIN_DISTINCT = 0, MC_RETAIN_LITERAL = 1, MC_RETAIN_TOPK = 2 } mc_retain_mode;

/* Which layer of the pair a call restores / attends for. BOTH = the two layers at once
 * (two query sets, one pass over the shared directions). */
typedef enum { MC_LAYER_LM1 = 0, MC_LAYER_L = 1, MC_LAYER_BOTH = 2 } mc_layer_sel;

/* Operations whose scratch need mc_workspace_bytes reports. */
typedef enum { MC_OP_MERGE = 0, MC_OP_DECODE_ATTN = 1 } mc_op;

/* The merge function.  MC_MERGE_SLERP is the method (Eq. 3, both magnitudes kept).  The other two
 * are the alternatives the paper compares it with: they merge the two rows into ONE vector that
 * stands for both layers -- MC_MERGE_FMAX the direction of the mean times the larger of the two
 * magnitudes (Appendix, "maximum norm-preserving interpolation"), MC_MERGE_MEAN the plain average
 * (Sec. 3.1) -- stored in the same format (direction, the one magnitude for both layers), so restore
 * and attention do not change.  The angular distance and the retention are the same for all three;
 * t is used by MC_MERGE_SLERP only. */
typedef enum mc_merge_fn { MC_MERGE_SLERP = 0, MC_MERGE_FMAX = 1, MC_MERGE_MEAN = 2 } mc_merge_fn;

/* Where the interpolation parameter of Eq. 3 comes from.  MC_T_FIXED: cfg->t for every token (the paper's
 * setting, t = 0.6).  MC_T_MAGNITUDE_RATIO: per token t_i = |x^l_i| / (|x^{l-1}_i| + |x^l_i|) -- Sec. 5's
 * ablation of t observes that the best t follows the relative magnitude ratio of adjacent layers and
 * suggests determining t from it; the formula is our reading (the longer row pulls the direction its
 * way, equal lengths give the geodesic midpoint).  cfg->t is then ignored. */
typedef enum mc_t_mode { MC_T_FIXED = 0, MC_T_MAGNITUDE_RATIO = 1 } mc_t_mode;

/* Status word indices (mc_read_status). */
enum {
  MC_STATUS_FLAGS = 0,          /* bit 0: retained pool overflow; bit 1: a bounded wait ran out;
                                   bit 2: a length or page id outside the declared bounds was met;
                                   bit 3: a range check of the range-checked build failed;
                                   bit 4: mc_prefill_merge_pair's distance hint was too high */
  MC_STATUS_RETAINED_TOTAL = 1, /* retained entries the last merge selected (K and V segments together) */
  MC_STATUS_NEAR_THRESHOLD = 2, /* tokens of the last merge whose distance lies within 1e-6 of their segment's
                                   retention threshold (a differently rounded d could have decided them the
                                   other way) */
  MC_STATUS_RESERVED1 = 3,
  MC_STATUS_WORDS = 4
};
#define MC_FLAG_RETAIN_OVERFLOW 1
#define MC_FLAG_WAIT_TIMEOUT 2
/* A kernel met a seq_lens entry outside [0, max_seq_len] or a page id outside [0, n_pages) (or a
 * token position past max_pages_per_seq pages).  Such a value is never turned into an address: the
 * length is clamped, the page's rows are not written (merge, restore, append) or page 0 is read in
 * its place (decode attention: the result of that sequence is then meaningless). */
#define MC_FLAG_BAD_METADATA 4
/* Range-checked build only (mc_build_flags() & MC_BUILD_BOUNDS): an index the library derived from the
 * pair cache's own contents -- a retained entry's token index, a retained range against the pool's
 * capacity, a compaction slot -- fell outside its bounds.  The access is skipped, the kernel carries
 * on, results that depended on it are meaningless. */
#define MC_FLAG_BOUNDS 8
/* mc_prefill_merge_pair: a segment's retention threshold fell below the caller's distance hint, so the raw
 * layer-l row of some retained token may not have been stored; merge that pair again with a lower hint. */
#define MC_FLAG_HINT_TOO_HIGH 16

/* Method parameters and tensor geometry (Sec. 4.1-4.2, Sec. 5 defaults t = 0.6, gamma = 0.05). */
typedef struct mc_config {
  int32_t n_kv_heads;  /* kv heads per layer */
  int32_t n_q_heads;   /* query heads; n_q_heads / n_kv_heads must be 1, 2, 4 or 8 (at most 4 with MC_LAYER_BOTH) */
  int32_t head_dim;    /* must be 128 */
  int32_t page_size;   /* tokens per page: 16, 32 or 64 */
  int32_t dtype;       /* mc_dtype of K/V/q/out storage */
  int32_t retain_mode; /* mc_retain_mode */
  double t;            /* interpolation parameter of Eq. 3: 0 -> direction of layer l-1, 1 -> of layer l */
  double gamma;        /* retention threshold of Eq. 4 */
  int32_t merge_fn;    /* mc_merge_fn: how the two rows of a token become the shared row */
  int32_t cache_bits;  /* storage of the shared directions E: 0 or 16 = the 16-bit type `dtype`; 4 = the 4-bit
                          shared cache described at mc_pair_cache (page_size must then be 32) */
  int32_t t_mode;      /* mc_t_mode: where Eq. 3's t comes from */
  int32_t retain_union; /* 0: Eq. 4 applied to keys and values separately (Algorithm 2 computes I_k and I_v);
                           1: one set per (sequence, head), the union of the two (Sec. 4.2 writes the pair cache
                           with a single I): a token either rule keeps is kept unmerged in both tensors.
                           Not with MC_RETAIN_TOPK. */
  int32_t append_slack; /* retention of tokens appended during decode (Sec. 4.2 keeps "unmergeable" tokens; Algorithm 2
                           decides only over the prefill tokens, so this is an extension).  0: an appended token is
                           always merged.  n > 0: every segment's retained list is laid out with n free entries
                           behind it when the pair is merged, and mc_append_pair applies Eq. 4 to the new token
                           with the segment's stored d_min and d_max (the threshold of the prefill tokens,
                           never recomputed): a token it keeps takes the next free entry.  Threshold modes only
                           (with MC_RETAIN_TOPK appended tokens are always merged); gamma = 0 keeps nothing. */
} mc_config;

/* Batch geometry shared by the layer pools and the pair cache. */
typedef struct mc_batch {
  const int32_t* block_table; /* [batch][max_pages_per_seq] page ids; entries past a sequence's pages are ignored */
  const int32_t* seq_lens;    /* [batch] cached tokens per sequence */
  int32_t batch;
  int32_t max_pages_per_seq;
  int32_t max_seq_len;        /* host-known upper bound of seq_lens (sizes grids and workspaces) */
  int32_t reserved;
  int64_t n_pages;            /* pages in every pool */
} mc_batch;

/* One layer's K and V pools: [n_pages][n_kv_heads][page_size][128], 16-bit. */
typedef struct mc_layer_kv {
  void* k_pool;
  void* v_pool;
} mc_layer_kv;

/* One layer's K and V stored in 4 bits (Sec. 5: MiniCache on top of 4-bit KIVI quantisation; the
 * paper names the scheme only, the layout is ours).  Asymmetric round-to-nearest, groups of 32:
 * value = code * scale + zero, scale and zero in binary16.  page_size must be 32 (one key group =
 * the page's tokens).
 * k_codes, v_codes  [n_pages][n_kv_heads][page_size][64] bytes; channel 2i in the low, 2i+1 in the high nibble of byte i
 * k_meta            [n_pages][n_kv_heads][128][2] binary16 (scale, zero): keys are quantised per channel,
 *                   a group = the 32 tokens of the page
 * v_meta            [n_pages][n_kv_heads][page_size][4][2] binary16: values per token, a group = 32 channels
 * All four 256-byte aligned. */
typedef struct mc_layer_q4 {
  const void* k_codes;
  const void* k_meta;
  const void* v_codes;
  const void* v_meta;
} mc_layer_q4;

/* The shared cache C^{l,l-1} of one layer pair (Sec. 4.2: [E, R^l, R^{l-1}, |X^{l-1}|, |X^l|, I]).
 *
 * e_k / e_v  [n_pages][n_kv_heads][tile] bytes, tile = page_size * 256 + 2 * page_size * 4 bytes: the
 *            shared directions E of one (page, head) -- page_size rows of 128 values of the 16-bit
 *            storage type, every token position kept -- followed by the two layers' scales
 *            [2][page_size] fp32 ([0]: layer l-1, [1]: layer l).  Inside a row the sixteen 16-byte
 *            chunks are permuted: chunk c of row r is stored at chunk position
 *            (c & 8) | ((c & 7) ^ (r & 7)), the order the attention kernel wants in shared memory.
 *            A scale is |x| / |e_stored|, the magnitude of Eq. 2 already divided by the length of
 *            the rounded direction, so that restore is one multiply: x_hat = e_stored * scale.
 *            The scales of a retained token are -0.0f (its rows are kept raw in ret_rows): a zero,
 *            so that the shared direction contributes nothing for it, whose sign marks the token.
 * dist       [n_pages][n_kv_heads][2][page_size] fp32 angular distance d = Omega / pi; slot 0: K, 1: V.
 * Retention, per segment seg = (tensor * batch + b) * n_kv_heads + head (tensor 0 = K, 1 = V):
 * ret_count  [2 * batch * n_kv_heads] retained tokens of the segment
 * ret_offset [2 * batch * n_kv_heads + 1] first slot of the segment: the exclusive prefix of ret_count, plus
 *            cfg->append_slack free entries behind every segment's list (their ret_index is -1 until
 *            mc_append_pair fills them); ret_capacity must cover those too
 * ret_index  [ret_capacity] token indices, ascending inside a segment
 * ret_rows   [2][ret_capacity][272 bytes]: [0] layer l-1, [1] layer l; an entry is the raw 16-bit row
 *            (256 bytes, a bit copy of the input), the token's index (int32) and 12 bytes of padding,
 *            so that a run of entries is one contiguous, 16-byte aligned block for a bulk copy
 * ret_prefix [2 * batch * n_kv_heads][ret_prefix_stride]: entry j = how many of the segment's retained
 *            tokens lie before token 128 * j (so a token range maps to a range of the segment's list
 *            without searching).  ret_prefix_stride (a host-side number, fixed when the pair is merged)
 *            must be at least ceil(max_seq_len at merge / 128) + 1.
 * seg_minmax [2 * batch * n_kv_heads][2] fp32 d_min, d_max of the prefill tokens
 * status     [MC_STATUS_WORDS] int32 */
typedef struct mc_pair_cache {
  void* e_k;  /* cache_bits = 4: the 4-bit tile pools, see below */
  void* e_v;
  float* dist;
  int32_t* ret_count;
  int32_t* ret_offset;
  int32_t* ret_index;
  void* ret_rows;
  int64_t ret_capacity;
  int32_t* ret_prefix;
  int64_t ret_prefix_stride;
  float* seg_minmax;
  int32_t* status;
  void* res_k; /* cache_bits = 4 only (else ignored, may be NULL): residual tiles, see below */
  void* res_v;
} mc_pair_cache;

/* The 4-bit shared cache (cfg->cache_bits = 4; Sec. 5: MiniCache on top of 4-bit KIVI quantisation --
 * the paper names the scheme only; the reading and the layout are ours).  The merged directions,
 * already rounded to the 16-bit type, are quantised page by page (page_size = 32 = the group size):
 * keys per channel (a group = the page's 32 tokens of one channel), values per token (a group = 32
 * consecutive channels), asymmetric round-to-nearest: scale = (max - min) / 15 and zero = min, both
 * kept in the 16-bit type (a constant group stores scale 1), code = clamp(rint((x - zero) / scale), 0, 15).
 * A stored direction element is code * scale + zero rounded ONCE to the 16-bit type; the scales of
 * Eq. 2 are |x| / |that stored direction|.  Only complete pages are quantised: the tokens of a
 * sequence's last, incomplete page stay in 16 bits (KIVI's full-precision residual) in the residual
 * tile of their (sequence, head) until mc_append_pair completes the page and quantises it.
 *
 * e_k / e_v  [n_pages][n_kv_heads][2816 bytes]; a tile = 2048 bytes of codes, 512 of group parameters,
 *            then the two layers' scales [2][32] fp32 as in the 16-bit tile.
 *   K codes  token row r at byte 64 r; in 32-bit word w of a row, bits [4p, 4p+4) hold channel 8w + 2p
 *            and bits [16 + 4p, 16 + 4p + 4) channel 8w + 2p + 1 (p = 0..3).
 *   K groups sixteen 16-byte chunks of scales, then sixteen of zeros (16-bit type); the chunk of the
 *            channels [8 o, 8 o + 8) sits at chunk position 4 (o & 3) + (o >> 2).
 *   V codes  sixteen 128-byte blocks, block i = tokens 2i and 2i+1; its 16-byte chunk c (0..7) sits at
 *            chunk position c ^ ((i & 3) << 1); in word k (0..3) of chunk c the low 16 bits belong to
 *            token 2i, the high 16 bits to token 2i+1, and bits [4n, 4n+4) of a half hold channel
 *            32 k + 16 (n >> 1) + 8 (n & 1) + c (n = 0..3).
 *   V groups per token pair i 32 bytes: four words (scale of token 2i, scale of token 2i+1) for the
 *            channel groups 0..3, then four such words of zeros.
 *            (These orders are the ones in which the attention kernel builds tensor-core fragments
 *            straight from the codes.)
 * res_k / res_v  [batch][n_kv_heads][8448 bytes]: one 16-bit tile (the format of cfg->cache_bits = 16,
 *            page_size 32) per (sequence, head) holding the tokens [32 floor(n / 32), n).
 * dist, the retention fields and status are as for the 16-bit cache. */

/* Byte sizes of the buffers of one mc_pair_cache (Sec. 4.2: the shared cache C of a layer pair) for
 * cfg, batch->batch, batch->n_pages, batch->max_seq_len (the longest sequence at merge time) and a
 * retained-row pool of ret_capacity entries.  e_bytes is the size of e_k and of e_v alike. */
typedef struct mc_pair_sizes {
  size_t tile_bytes;        /* one (page, head) tile of e_k / e_v */
  size_t e_bytes;
  size_t dist_bytes;
  size_t ret_count_bytes;
  size_t ret_offset_bytes;
  size_t ret_index_bytes;
  size_t ret_rows_bytes;
  size_t ret_prefix_bytes;
  size_t seg_minmax_bytes;
  size_t status_bytes;
  int64_t ret_prefix_stride; /* value for mc_pair_cache.ret_prefix_stride */
  size_t total_bytes;        /* all buffers, each rounded up to 256 bytes */
  size_t res_bytes;          /* res_k and res_v alike; 0 unless cfg->cache_bits = 4 */
} mc_pair_sizes;

/* What the last merge into a pair did (Sec. 4.2 retention, Sec. 4.3 footprint). */
typedef struct mc_stats {
  int32_t flags;            /* MC_STATUS_FLAGS */
  int32_t reserved;
  int64_t retained_total;   /* retained entries, K and V segments together */
  int64_t near_threshold;   /* tokens with |d - threshold| < 1e-6 (MC_STATUS_NEAR_THRESHOLD) */
  int64_t token_heads;      /* (token, kv head) rows per layer and tensor = sum(seq_lens) * n_kv_heads */
  int64_t full_bytes;       /* the two layers' K and V uncompressed: 4 * token_heads * 256 */
  int64_t compressed_bytes; /* first-principles size of the shared cache: per (token, head, tensor) one
                               direction row, two magnitudes and the distance; per retained entry both raw
                               rows and the index (Sec. 4.3 counts the same items) */
  int64_t stored_bytes;     /* what the pair occupies in this library's layout: whole tiles of the pages in
                               use, padded retained entries, per-segment tables */
} mc_stats;

/* Pure host arithmetic; no device work.  (The paper has no counterpart: buffer planning.) */
mc_status mc_pair_bytes(const mc_config* cfg, const mc_batch* batch, int64_t ret_capacity, mc_pair_sizes* out);

/* Reads the pair's status words and the batch's lengths after synchronising `stream` and fills `out`.
 * Returns like mc_read_status (MC_ERR_CAPACITY / MC_ERR_DEVICE_STATUS when a flag is set; `out` is
 * filled either way).  batch->seq_lens must be the lengths the pair was merged at for the byte
 * counts to describe that merge. */
mc_status mc_get_stats(const mc_config* cfg, const mc_batch* batch, const mc_pair_cache* pair, void* stream,
                       mc_stats* out);

/* Library version (major * 10000 + minor * 100 + patch). No device work. */
int32_t mc_version(void);

/* How the library was built (the paper has no counterpart).  MC_BUILD_BOUNDS: compiled with -DMC_BOUNDS=1,
 * the debugging build in which the kernels also range-check every index they derive from the pair cache's
 * contents (see MC_FLAG_BOUNDS); it stands in for a memory checker where none can be run.  Checks of the
 * caller's batch description (MC_FLAG_BAD_METADATA) are part of every build. */
#define MC_BUILD_BOUNDS 1
int32_t mc_build_flags(void);

/* Human-readable name of a status code (static string). */
const char* mc_status_str(int32_t status);

/* Text of the last CUDA error seen by this thread inside the library ("" if none). */
const char* mc_last_cuda_error(void);

/* Scratch bytes `op` needs for this geometry (a multiple of 256).  Pure host arithmetic.
 * `n_query_sets` is 2 for MC_LAYER_BOTH decode attention, else 1 (ignored for MC_OP_MERGE).
 * With cfg->cache_bits = 4 the merge scratch also holds the 16-bit direction tiles of both tensors
 * before they are quantised (2 * n_pages * n_kv_heads * 8448 bytes: batch->n_pages must be set). */
mc_status mc_workspace_bytes(const mc_config* cfg, const mc_batch* batch, int32_t op,
                             int32_t n_query_sets, size_t* bytes);

/* Algorithm 2 "MiniCache Prefill" for one layer pair: Eq. 3 merge of every cached token of
 * every sequence (K and V), magnitudes (Eq. 2), distances, and -- if do_retention -- the
 * retention set of Eq. 4 with the raw rows of both layers gathered into `out`.
 * lm1 / l : the two layers' pools (read only; they may be released once the stream has run
 *           the call).  out: all fields written; status words are cleared first.
 * With do_retention == 0 every ret_count is set to 0.
 * If the selection needs more than ret_capacity entries the overflow flag is set, no retained
 * entry is written and every ret_count is 0 (the merged directions are still valid).
 * workspace: at least mc_workspace_bytes(MC_OP_MERGE) bytes, 256-byte aligned, contents
 * irrelevant on entry, must stay untouched until the call has run on the stream.
 * cfg->cache_bits = 4: the merged directions are formed and rounded to cfg->dtype exactly as for the
 * 16-bit cache (in the workspace), retention marks its tokens, then every complete page is quantised
 * into out->e_k / e_v and each sequence's last, incomplete page is copied to out->res_k / res_v. */
mc_status mc_merge_pair(const mc_config* cfg, const mc_batch* batch, const mc_layer_kv* lm1,
                        const mc_layer_kv* l, const mc_pair_cache* out, int32_t do_retention,
                        void* workspace, size_t workspace_bytes, void* stream);

/* Algorithm 1's prefill loop over the merged half of the model ("for l = S .. L-1: if l is odd, merge
 * layers l and l-1"): mc_merge_pair for n_pairs layer pairs of one batch at once.  lm1[i], l[i], out[i]
 * are pair i's layers and pair cache (host arrays of pointers, read before the call returns; every pair
 * needs its own pair cache).  The pairs are independent, so their rows are streamed by one persistent grid
 * and their segments go through one retention pass: four launches for up to 8 pairs instead of four per
 * pair.  Results are bit-identical to n_pairs calls of mc_merge_pair.
 * workspace: n_pairs * mc_workspace_bytes(MC_OP_MERGE) bytes, 256-byte aligned.
 * A length outside its declared bound or a wait that ran out is recorded in the status words of the first
 * pair of its group of 8; everything else in the pair's own.  cfg->cache_bits = 4 is not supported here
 * (MC_ERR_UNSUPPORTED): merge such pairs one by one. */
mc_status mc_merge_pairs(const mc_config* cfg, const mc_batch* batch, int32_t n_pairs,
                         const mc_layer_kv* const* lm1, const mc_layer_kv* const* l,
                         const mc_pair_cache* const* out, int32_t do_retention, void* workspace,
                         size_t workspace_bytes, void* stream);

/* Admission of new sequences into a running batch (Algorithm 1's prefill branch for sequences that arrive
 * while others decode; the paper's serving experiment, Sec. 5, gets its throughput from the larger live
 * batch): Algorithm 2 "MiniCache Prefill" for the sequences [seq_begin, seq_begin + seq_count) of the batch
 * only, for n_pairs layer pairs in one launch sequence.  The other sequences' tiles, tables and retained
 * entries are not touched, so the call may run on a second stream while decode steps attend them -- as
 * long as the admitted sequences' seq_lens entries read 0 for those decode calls (give this call a
 * mc_batch whose seq_lens holds the new lengths, and copy them into the decode batch's seq_lens once this
 * call has run).
 * lm1 / l            16-bit layers per pair, or both NULL with q4_lm1 / q4_l given (4-bit layers, page 32)
 * rows_per_seq       the retained pool is used as one region per sequence: sequence b owns the entries
 *                    [b * rows_per_seq, (b + 1) * rows_per_seq) (batch->batch * rows_per_seq <= ret_capacity).
 *                    A sequence whose retention needs more keeps nothing and MC_FLAG_RETAIN_OVERFLOW is set.
 *                    A pair cache filled this way must be filled this way for all its sequences (never mix
 *                    with mc_merge_pair, whose retained lists are one compact run for the whole batch).
 * Status words are not cleared (flags accumulate); MC_STATUS_RETAINED_TOTAL / NEAR_THRESHOLD are not kept.
 * workspace          n_pairs * mc_workspace_bytes(MC_OP_MERGE) bytes (with cfg->cache_bits = 4: the part
 *                    without the staging tiles per pair, plus the staging tiles once), 256-byte aligned. */
mc_status mc_admit_sequences(const mc_config* cfg, const mc_batch* batch, int32_t seq_begin, int32_t seq_count,
                             int32_t n_pairs, const mc_layer_kv* const* lm1, const mc_layer_kv* const* l,
                             const mc_layer_q4* const* q4_lm1, const mc_layer_q4* const* q4_l,
                             const mc_pair_cache* const* out, int64_t rows_per_seq, int32_t do_retention,
                             void* workspace, size_t workspace_bytes, void* stream);

/* The K/V projection of layer l (the stand-in for the model's own: the library computes K^l = X W_k^T and
 * V^l = X W_v^T itself so that it can merge in the projection's epilogue).
 * x        [batch * x_seq_stride][d_model] hidden states entering layer l's K/V projection, cfg->dtype;
 *          token i of sequence b is row b * x_seq_stride + i; x_seq_stride a multiple of 128, >= max_seq_len
 * w_k, w_v [n_kv_heads * 128][d_model] cfg->dtype: row (head * 128 + channel) holds that output channel's
 *          weights (the transposed weight matrix, contiguous along d_model)
 * d_model  a multiple of 64.  All three base addresses 256-byte aligned. */
typedef struct mc_projection {
  const void* x;
  const void* w_k;
  const void* w_v;
  int32_t d_model;
  int32_t x_seq_stride;
} mc_projection;

/* Algorithm 1's prefill branch with the merge fused into layer l's projection ("merge at odd layers during
 * prefill"): layer l's K and V rows are formed on chip (tensor cores, fp32 accumulation, rounded once to
 * cfg->dtype -- the rows the model would have cached) and merged with layer l-1's cached rows (lm1) by
 * Eq. 2 / Eq. 3 right there, so they are never written to and read back from device memory; `out` receives
 * exactly what mc_merge_pair would have written for those rows.
 * Retention (Eq. 4) needs the raw layer-l rows of the tokens it keeps, and which tokens those are is known
 * only once every distance of a segment is: the rows of tokens with distance d > d_hint are therefore also
 * stored, at their places in the pools `l` (everything else in `l` is left untouched), and the retention
 * pass gathers from there.  d_hint < 0 stores every row (`l` then holds the whole layer, e.g. for checking).
 * If a segment's threshold turns out below d_hint, MC_FLAG_HINT_TOO_HIGH is set: merge that pair again with
 * a lower hint.  With do_retention == 0 nothing needs to be stored (pass d_hint = 2).
 * Limits: cfg->merge_fn = MC_MERGE_SLERP, cfg->retain_mode = MC_RETAIN_DISTINCT (or d_hint < 0), 16-bit
 * shared cache, d_model % 64 == 0.  workspace as for mc_merge_pair. */
mc_status mc_prefill_merge_pair(const mc_config* cfg, const mc_batch* batch, const mc_projection* proj,
                                const mc_layer_kv* lm1, const mc_layer_kv* l, const mc_pair_cache* out,
                                float d_hint, int32_t do_retention, void* workspace, size_t workspace_bytes,
                                void* stream);

/* mc_merge_pair for layers stored in 4 bits: the rows are de-quantised inside the merge kernel
 * (code * scale + zero in fp32) and merged exactly as in mc_merge_pair; the pair cache it writes is
 * the same 16-bit format (cfg->dtype).  The raw rows of retained tokens are the de-quantised values
 * rounded once to cfg->dtype.  cfg->page_size must be 32. */
mc_status mc_merge_pair_q4(const mc_config* cfg, const mc_batch* batch, const mc_layer_q4* lm1,
                           const mc_layer_q4* l, const mc_pair_cache* out, int32_t do_retention,
                           void* workspace, size_t workspace_bytes, void* stream);

/* Algorithm 2 "MiniCache Decoding", the branch that compresses the step's new token pair:
 * merges k/v_new_lm1 with k/v_new_l ([batch][n_kv_heads][128], 16-bit) by Eq. 3 and writes
 * direction, scales and distance at token position seq_lens[b] of every sequence (the block
 * table must already hold a page for it).  With cfg->append_slack == 0 no retention decision is taken
 * for new tokens.  With cfg->append_slack > 0 (the value the pair was merged with) a new token whose
 * distance passes Eq. 4 against the segment's stored d_min, d_max (both tensors' rules with
 * cfg->retain_union) is kept unmerged: its two raw rows go to the next free entry of the segment's
 * retained list, its scales become -0.0, ret_count, ret_prefix and the retained total are updated.  A
 * segment whose free entries are used up sets MC_FLAG_RETAIN_OVERFLOW and the token is merged instead.
 * seq_lens is not modified: the caller advances it once all layers of the step are done.
 * cfg->cache_bits = 4: the row goes to slot seq_lens[b] % 32 of the sequence's residual tile; when
 * that fills the page (slot 31) the same kernel quantises the 32 rows into the page's 4-bit tile. */
mc_status mc_append_pair(const mc_config* cfg, const mc_batch* batch, const mc_pair_cache* pair,
                         const void* k_new_lm1, const void* v_new_lm1, const void* k_new_l,
                         const void* v_new_l, void* stream);

/* Eq. 2 + Sec. 4.2 "Cache restoration": writes the dense restored K and V of one layer
 * (layer_sel = MC_LAYER_LM1 or MC_LAYER_L) into dst pools of the same paged layout:
 * x_hat = e * scale, then retained rows overwritten with their raw copies.
 * dst_fp32 == 0: dst pools hold cfg->dtype (the product is rounded once to it).
 * dst_fp32 != 0: dst pools are [n_pages][n_kv_heads][page_size][128] binary32: the product as
 *                computed, raw rows converted exactly.
 * cfg->cache_bits = 4: e is the stored direction of the 4-bit cache (code * scale + zero rounded once
 * to cfg->dtype) for tokens in complete pages and the residual tile's row for the others. */
mc_status mc_restore(const mc_config* cfg, const mc_batch* batch, const mc_pair_cache* pair,
                     int32_t layer_sel, const mc_layer_kv* dst, int32_t dst_fp32, void* stream);

/* Algorithm 2 "MiniCache Decoding": single-query attention of every sequence over the restored
 * cache of one layer, computed straight from the compressed pair (restore fused; the dense K/V
 * is never materialised), split along the token axis and combined by log-sum-exp.
 * layer_sel   MC_LAYER_LM1 / MC_LAYER_L: one query set.  MC_LAYER_BOTH: two query sets, set 0
 *             attends layer l-1 and set 1 layer l, sharing one pass over the directions.
 * q           [n_sets][batch][n_q_heads][128] 16-bit
 * k_new,v_new [n_sets][batch][n_kv_heads][128] 16-bit raw rows of the step's new token, attended
 *             as one extra token after the cached ones; both NULL to attend the cache alone.
 * sm_scale    multiplies q.k before the softmax (Algorithm 2 prints none; pass 1/sqrt(128)).
 * out         [n_sets][batch][n_q_heads][128] 16-bit
 * lse         [n_sets][batch][n_q_heads] fp32 natural-log sum of exponentials, or NULL
 * workspace   at least mc_workspace_bytes(MC_OP_DECODE_ATTN, n_sets) bytes, 256-byte aligned.
 * A sequence with seq_lens[b] == 0 and no new token yields zeros (lse = -inf).
 * cfg->cache_bits = 4: the 4-bit tiles are streamed as they are and de-quantised in registers (one
 * packed 16-bit FMA per element pair gives the stored direction exactly); the residual tile of a
 * sequence's last page is attended in 16 bits.  Same arguments, same workspace size. */
mc_status mc_decode_attn(const mc_config* cfg, const mc_batch* batch, const mc_pair_cache* pair,
                         int32_t layer_sel, const void* q, const void* k_new, const void* v_new,
                         float sm_scale, void* out, float* lse, void* workspace,
                         size_t workspace_bytes, void* stream);

/* One decode step of a layer pair's second layer in one call (Algorithm 2 "MiniCache Decoding": attend, then
 * compress the step's token pair): mc_decode_attn with the first ten arguments, followed by mc_append_pair with
 * k/v_new_lm1, k/v_new_l -- same results, bit for bit, as the two calls one after the other.  With a 16-bit
 * shared cache the append rides on the attention's second launch (a few more blocks of the combine kernel,
 * which run once the split kernel is complete) instead of taking a launch of its own; with cfg->cache_bits = 4
 * it is the two calls.  Typical use: layer_sel = MC_LAYER_L with k_new = k_new_l, v_new = v_new_l (the pair's
 * layer l-1 was attended by a plain mc_decode_attn before), or MC_LAYER_BOTH.  Every argument of both calls is
 * checked before anything is launched. */
mc_status mc_decode_attn_append(const mc_config* cfg, const mc_batch* batch, const mc_pair_cache* pair,
                                int32_t layer_sel, const void* q, const void* k_new, const void* v_new,
                                float sm_scale, void* out, float* lse, const void* k_new_lm1,
                                const void* v_new_lm1, const void* k_new_l, const void* v_new_l,
                                void* workspace, size_t workspace_bytes, void* stream);

/* Host-buffer form of mc_merge_pair (Algorithm 2 "MiniCache Prefill" with the layers' K/V arriving
 * from the host): host_lm1 / host_l are HOST pools (pinned memory for asynchronous copies) in the
 * paged layout; they are copied into the caller's device pools dev_lm1 / dev_l on `stream`
 * (n_pages * n_kv_heads * page_size * 256 bytes each) and merged there.  Nothing is allocated. */
mc_status mc_merge_pair_host(const mc_config* cfg, const mc_batch* batch, const mc_layer_kv* host_lm1,
                             const mc_layer_kv* host_l, const mc_layer_kv* dev_lm1,
                             const mc_layer_kv* dev_l, const mc_pair_cache* out, int32_t do_retention,
                             void* workspace, size_t workspace_bytes, void* stream);

/* Host-buffer form of mc_decode_attn (Algorithm 2 "MiniCache Decoding" for a caller whose queries
 * live on the host): q_host, k_new_host, v_new_host are read from and out_host (and lse_host, if not
 * NULL) written to HOST memory, through `dev_io`, a device staging buffer of at least
 * mc_decode_io_bytes() bytes (256-byte aligned).  The copies are enqueued on `stream` around the
 * kernels; out_host is valid once the stream has run the call.  Nothing is allocated. */
mc_status mc_decode_attn_host(const mc_config* cfg, const mc_batch* batch, const mc_pair_cache* pair,
                              int32_t layer_sel, const void* q_host, const void* k_new_host,
                              const void* v_new_host, float sm_scale, void* out_host, float* lse_host,
                              void* dev_io, size_t dev_io_bytes, void* workspace,
                              size_t workspace_bytes, void* stream);

/* Stages the inputs of later mc_decode_attn / mc_decode_attn_append calls from HOST memory: copies q
 * ([n_query_sets][batch][n_q_heads][128]) and, if given, k_new / v_new ([n_query_sets][batch][n_kv_heads][128])
 * into `dev_io` (device memory of at least mc_decode_io_bytes(n_query_sets) bytes, 256-byte aligned) on `stream`
 * and returns where they landed in *q_dev, *k_new_dev, *v_new_dev (device pointers into dev_io; set k of a
 * two-set staging starts n_q_heads (n_kv_heads) * batch * 256 bytes after set 0).  Meant to be issued on a second
 * stream, a call or a layer pair ahead of the attention that consumes the rows, so that the transfer -- slow when the
 * host link is busy with an upload -- is off the decode loop's critical path; the caller orders the two streams
 * (an event after the staging, one after the attention before the buffer is staged again).  Pinned,
 * device-addressable host memory is read by a kernel, any other by asynchronous copies.  An attention call can
 * write its result straight to pinned host memory: pass the buffer's device pointer as `out`. */
mc_status mc_decode_stage_host(const mc_config* cfg, const mc_batch* batch, int32_t n_query_sets,
                               const void* q_host, const void* k_new_host, const void* v_new_host,
                               void* dev_io, size_t dev_io_bytes, void** q_dev, void** k_new_dev,
                               void** v_new_dev, void* stream);

/* The other direction: copies the result of an attention call ([n_query_sets][batch][n_q_heads][128] 16-bit, and the
 * log-sum-exps [n_query_sets][batch][n_q_heads] fp32 if lse_dev / lse_host are given -- both or neither) from device
 * memory to HOST memory, asynchronously on `stream` (the device-to-host copy engine: it does not compete with an
 * upload).  Meant for a stream of its own, ordered after the attention by the caller, so that the transfer is off
 * the decode loop's critical path. */
mc_status mc_decode_drain_host(const mc_config* cfg, const mc_batch* batch, int32_t n_query_sets,
                               const void* out_dev, const float* lse_dev, void* out_host, float* lse_host,
                               void* stream);

/* Bytes of device staging mc_decode_attn_host needs (q, new K/V rows, out, lse). Host arithmetic. */
mc_status mc_decode_io_bytes(const mc_config* cfg, const mc_batch* batch, int32_t n_query_sets,
                             size_t* bytes);

/* Largest split-partial scratch mc_decode_attn_static can serve (bytes of its built-in array). */
#define MC_STATIC_SCRATCH_BYTES (8u * 1024u * 1024u)

/* mc_decode_attn without a workspace argument.  (The paper has no counterpart: this exists for
 * integration reasons only.)  Some callers cannot hand the library scratch memory: a serving
 * engine that has already given every free byte of HBM to its KV-cache pool, a plugin that is
 * only passed its input and output tensors, or a decode loop that must not call cudaMalloc
 * because an allocation synchronises the device and stalls every stream.  For them the split
 * partials live in an array that is part of the library image: MC_STATIC_SCRATCH_BYTES of device
 * memory on every GPU that loads the library, held until the process exits.
 *
 * Arguments, results and numerics are those of mc_decode_attn (same kernels).  Differences:
 * - A geometry whose partials need more than MC_STATIC_SCRATCH_BYTES (what
 *   mc_workspace_bytes(MC_OP_DECODE_ATTN) reports) is refused with MC_ERR_CAPACITY before anything
 *   is launched; mc_last_cuda_error() then names both sizes.
 * - The first call on each device looks up the array's device address (one runtime query, no
 *   allocation).  Make that first call outside any stream capture.  The array used is the one of
 *   the device that is current when the call is made: `stream` must belong to that device.
 * - All calls on a device share the one array.  Nothing in it has to start at zero: every slot a
 *   call reads was written earlier by the same call.  But two calls that may run at the same time
 *   on the GPU (different streams, no ordering between them) overwrite each other's partials:
 *   order them on one stream or with events.
 * The call allocates and frees nothing, on the device or through any library. */
mc_status mc_decode_attn_static(const mc_config* cfg, const mc_batch* batch, const mc_pair_cache* pair,
                                int32_t layer_sel, const void* q, const void* k_new, const void* v_new,
                                float sm_scale, void* out, float* lse, void* stream);

/* Self-test of the error path of the bounded waits (the paper has no counterpart): enqueues a
 * one-warp kernel that waits, with the same bounded wait the streaming kernels use and a limit of
 * `poll_limit` polls, on a barrier that nothing completes.  The wait gives up, sets
 * MC_FLAG_WAIT_TIMEOUT in the pair's status words and the kernel returns normally: the context
 * stays usable and mc_read_status reports MC_ERR_DEVICE_STATUS until the next merge into the pair
 * clears the words. */
mc_status mc_selftest_wait_timeout(const mc_pair_cache* pair, int32_t poll_limit, void* stream);

/* Copies the pair's status words to host memory `out_words[MC_STATUS_WORDS]` after synchronising
 * `stream`.  Returns MC_ERR_CAPACITY if the overflow flag is set, MC_ERR_DEVICE_STATUS for any
 * other flag, MC_OK otherwise. */
mc_status mc_read_status(const mc_pair_cache* pair, void* stream, int32_t* out_words);

#ifdef __cplusplus
}
#endif
#endif /* MINICACHE_H_ */
