// Work items of the streaming kernels that walk every cached row of a batch (merge, restore): 64
// consecutive rows of one page.  The rows of a page are [head][token], so an item is one contiguous
// block in a layer pool, and a run of whole (page, head) tiles in the pair cache.
#pragma once
#include "mc_common.cuh"

namespace mc {

constexpr int kMaxBatchPages = 1024;  // sequences whose page-count prefix fits the kernels' shared memory

struct PageItem {
  int tensor, b, pslot, grp;
  int pg;  // page slot counted over the used pages of all sequences
};

// Sequence lengths and the exclusive prefix of the sequences' page counts into shared memory
// (len_s [batch], pre_s [batch + 1]); called by every thread of the CTA, ends with a barrier.
// Lengths above the declared bound are clamped to it (and flagged in `status`).
__device__ __forceinline__ void page_prefix(const Geom& g, int* len_s, int* pre_s, int n_threads, int32_t* status) {
  const int tid = threadIdx.x, lane = tid & 31;
  for (int b = tid; b < g.batch; b += n_threads) len_s[b] = checked_len(g, b, status);
  __syncthreads();
  if (tid < 32) {
    // a lane sums a run of sequences, the runs are scanned with shuffles
    const int ps = g.page_size;
    const int per = (g.batch + 31) / 32;
    const int b0 = min(lane * per, g.batch), b1 = min(b0 + per, g.batch);
    int sum = 0;
    for (int b = b0; b < b1; ++b) sum += (len_s[b] + ps - 1) >> g.page_shift;
    int incl = sum;
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) {
      const int v = __shfl_up_sync(0xffffffffu, incl, o);
      if (lane >= o) incl += v;
    }
    int acc = incl - sum;
    for (int b = b0; b < b1; ++b) {
      pre_s[b] = acc;
      acc += (len_s[b] + ps - 1) >> g.page_shift;
    }
    if (lane == 31) pre_s[g.batch] = incl;
  }
  __syncthreads();
}

// Only pages that hold tokens are enumerated: `pre` is the exclusive prefix of the sequences' page
// counts (pre[batch] = P, all of them), an item index is ((tensor * P) + pg) * items_per_page + grp
// -- row group fastest, then page, sequence, tensor.  A CTA walks its items with a fixed stride, so
// the decomposition is kept incrementally (no divisions per item) and the sequence is found by
// stepping forward in `pre`.  `tensor` runs over n_slots tensors (K and V of one pair, or of several
// pairs one after the other: slot = 2 * pair + tensor); tensor == n_slots marks the end.
__device__ __forceinline__ void page_item_init(PageItem& m, long long i, int ipp, int P, const int* pre, int n_slots = 2) {
  const long long per_tensor = (long long)P * ipp;
  if (P == 0 || i >= n_slots * per_tensor) {
    m.tensor = n_slots;
    m.b = m.pslot = m.grp = m.pg = 0;
    return;
  }
  m.tensor = (int)(i / per_tensor);
  const int rem = (int)(i - m.tensor * per_tensor);
  m.pg = rem / ipp;
  m.grp = rem - m.pg * ipp;
  m.b = 0;
  while (m.pg >= pre[m.b + 1]) ++m.b;
  m.pslot = m.pg - pre[m.b];
}
__device__ __forceinline__ void page_item_advance(PageItem& m, int s_pg, int s_grp, int ipp, int P, const int* pre,
                                                  int n_slots = 2) {
  if (m.tensor >= n_slots) return;
  m.grp += s_grp;
  const int carry = m.grp >= ipp ? 1 : 0;
  m.grp -= carry * ipp;
  m.pg += s_pg + carry;
  while (m.pg >= P) {
    m.pg -= P;
    m.b = 0;
    if (++m.tensor >= n_slots) return;
  }
  while (m.pg >= pre[m.b + 1]) ++m.b;
  m.pslot = m.pg - pre[m.b];
}

}  // namespace mc
