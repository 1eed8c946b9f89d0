// Shared device/host helpers of the MiniCache CUDA path (sm_100a).
#pragma once

#include <cuda_bf16.h>
#include <cuda_fp16.h>
#include <cuda_runtime.h>
#include <stdint.h>

#include "minicache.h"

namespace mc {

constexpr int kHeadDim = 128;
constexpr int kRowBytes = kHeadDim * 2;  // one 16-bit row
constexpr int kRetEntryBytes = 272;      // retained entry: raw 16-bit row, int32 token index, 12 bytes of padding
constexpr float kInvPi = 0.31830988618379067154f;

// Host-side launch plumbing ---------------------------------------------------
void set_cuda_error(cudaError_t e, const char* where);
#define MC_CUDA_CHECK(expr)            \
  do {                                 \
    cudaError_t _e = (expr);           \
    if (_e != cudaSuccess) {           \
      ::mc::set_cuda_error(_e, #expr); \
      return MC_ERR_CUDA;              \
    }                                  \
  } while (0)

// Every kernel of the library is launched with programmatic dependent launch allowed and begins
// with grid_dep_wait(): its blocks may be placed on the SMs while the previous kernel of the stream
// drains, but touch no memory before that kernel has completed.  grid_dep_launch() right after lets
// the next kernel do the same.  This removes the launch gap between the many short kernels of a
// merge and of a decode step.
template <typename... KArgs, typename... Args>
inline cudaError_t launch_pdl(void (*kernel)(KArgs...), dim3 grid, dim3 block, size_t smem, cudaStream_t stream,
                              Args... args) {
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = grid;
  cfg.blockDim = block;
  cfg.dynamicSmemBytes = smem;
  cfg.stream = stream;
  cudaLaunchAttribute attr[1];
  attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  attr[0].val.programmaticStreamSerializationAllowed = 1;
  cfg.attrs = attr;
  cfg.numAttrs = 1;
  return cudaLaunchKernelEx(&cfg, kernel, static_cast<KArgs>(args)...);
}
#if defined(__CUDACC__)
__device__ __forceinline__ void grid_dep_wait() { asm volatile("griddepcontrol.wait;" ::: "memory"); }
__device__ __forceinline__ void grid_dep_launch() { asm volatile("griddepcontrol.launch_dependents;" ::: "memory"); }
#endif

// Geometry handed to every kernel by value.
struct Geom {
  const int32_t* block_table;
  const int32_t* seq_lens;
  int batch;
  int max_pages_per_seq;
  int n_kv_heads;
  int page_size;
  int page_shift;  // log2(page_size)
  int max_seq_len;  // the caller's bound of seq_lens: longer lengths are clamped to it and flagged
  int n_pages;      // pages in every pool: page ids outside [0, n_pages) are never used as addresses
  // the sequences a merge works on: all of them, or (admission of new sequences into free slots) a
  // range; the others count as empty for that call
  int seq_begin, seq_count;
};

#if defined(__CUDACC__)
// The batch description is the caller's and may be stale or wrong.  No kernel ever turns an
// unchecked length or page id into an address: a length above the declared bound is clamped, a page
// id outside the pools is replaced by page 0 for reads and skips the write, and either sets
// MC_FLAG_BAD_METADATA in the pair's status words.
__device__ __forceinline__ int checked_len(const Geom& g, int b, int32_t* status) {
  if ((unsigned)(b - g.seq_begin) >= (unsigned)g.seq_count) return 0;  // not part of this call
  const int n = g.seq_lens[b];
  if (n < 0 || n > g.max_seq_len) {
    atomicOr(status, MC_FLAG_BAD_METADATA);
    return n < 0 ? 0 : g.max_seq_len;
  }
  return n;
}
__device__ __forceinline__ bool page_ok(const Geom& g, int page) { return (unsigned)page < (unsigned)g.n_pages; }
// Page id of page slot `slot` of sequence `b`; -1 (and the flag) if the slot or the id is out of range.
__device__ __forceinline__ int checked_page(const Geom& g, int b, int slot, int32_t* status) {
  if ((unsigned)slot < (unsigned)g.max_pages_per_seq) {
    const int page = g.block_table[(size_t)b * g.max_pages_per_seq + slot];
    if (page_ok(g, page)) return page;
  }
  atomicOr(status, MC_FLAG_BAD_METADATA);
  return -1;
}
#endif

// Range-checked build (-DMC_BOUNDS=1): indices derived from the pair cache's own contents are checked
// where they are used; a failed check records MC_FLAG_BOUNDS and the access is skipped.  In the normal
// build the check is the constant `true`.
#if defined(MC_BOUNDS) && MC_BOUNDS
#define MC_IN_BOUNDS(cond, status) ((cond) ? true : (atomicOr((status), MC_FLAG_BOUNDS), false))
#else
#define MC_IN_BOUNDS(cond, status) true
#endif

__host__ __device__ inline size_t align_up(size_t x, size_t a) { return (x + a - 1) / a * a; }

// Compressed tile of one (page, kv head, tensor) in the pair cache: page_size direction rows of
// 256 bytes, then the two layers' scales [2][page_size] fp32.  Inside a row the sixteen 16-byte
// chunks are permuted: chunk c of row r sits at position (c & 8) | ((c & 7) ^ (r & 7)).  A tile is
// thus one contiguous block that a single bulk copy brings into shared memory in a layout where
// eight consecutive rows of one chunk column fall into eight different bank groups (ldmatrix
// without conflicts), and the scales a layer needs arrive with it.
__host__ __device__ inline int tile_bytes(int page_size) { return page_size * kRowBytes + 2 * page_size * 4; }
__host__ __device__ inline int chunk_pos(int r, int c) { return (c & 8) | ((c & 7) ^ (r & 7)); }

// 16-bit storage types ---------------------------------------------------------
template <int DT>
struct Elem;
template <>
struct Elem<MC_F16> {
  // binary16 -> binary32 as x * 1 + 0 on the FMA pipe (sm_100 mixed-precision FMA); the plain
  // conversion instruction runs on the slow transcendental/conversion unit and was the
  // bottleneck of the merge kernel
  static __device__ __forceinline__ float2 unpack(uint32_t w) {
    float2 r;
    asm("{\n\t.reg .b16 lo, hi, one;\n\tmov.b32 {lo, hi}, %2;\n\tmov.b16 one, 0x3C00;\n\t"
        "fma.rn.f32.f16 %0, lo, one, 0f00000000;\n\tfma.rn.f32.f16 %1, hi, one, 0f00000000;\n\t}"
        : "=f"(r.x), "=f"(r.y)
        : "r"(w));
    return r;
  }
  static __device__ __forceinline__ uint32_t pack(float x, float y) {
    __half2 h = __floats2half2_rn(x, y);
    return *reinterpret_cast<uint32_t*>(&h);
  }
};
template <>
struct Elem<MC_BF16> {
  static __device__ __forceinline__ float2 unpack(uint32_t w) {
    // bfloat16 is the upper half of a binary32
    return make_float2(__uint_as_float(w << 16), __uint_as_float(w & 0xffff0000u));
  }
  static __device__ __forceinline__ uint32_t pack(float x, float y) {
    __nv_bfloat162 h = __floats2bfloat162_rn(x, y);
    return *reinterpret_cast<uint32_t*>(&h);
  }
};

// Streaming 16-byte global accesses (read once / write once data).
__device__ __forceinline__ uint4 ld_stream16(const void* p) {
  uint4 v;
  asm volatile("ld.global.nc.L1::no_allocate.v4.u32 {%0,%1,%2,%3}, [%4];"
               : "=r"(v.x), "=r"(v.y), "=r"(v.z), "=r"(v.w)
               : "l"(p));
  return v;
}
__device__ __forceinline__ void st_stream16(void* p, const uint4& v) {
  asm volatile("st.global.L1::no_allocate.v4.u32 [%0], {%1,%2,%3,%4};" ::"l"(p), "r"(v.x), "r"(v.y),
               "r"(v.z), "r"(v.w)
               : "memory");
}

// Sum over the 16 lanes that share one row (lane ^ 8, 4, 2, 1 stay inside a half-warp).
__device__ __forceinline__ float sum16(float v) {
  v += __shfl_xor_sync(0xffffffffu, v, 8);
  v += __shfl_xor_sync(0xffffffffu, v, 4);
  v += __shfl_xor_sync(0xffffffffu, v, 2);
  v += __shfl_xor_sync(0xffffffffu, v, 1);
  return v;
}

// Per-row scalars of the merge (Eq. 3 weights folded with 1/|x|, both magnitudes, distance).
struct RowScalars {
  float fa, fc;  // e = fa * a + fc * c
  float na, nc;  // |a|, |c|
  float d;       // Omega / pi
};

// Angle and SLERP weights from |a|^2, |c|^2, |u - v|^2, |u + v|^2 (u, v the unit directions).
// Omega = 2 atan2(|u - v|, |u + v|) is well conditioned at both ends of [0, pi], where arccos
// of a rounded cosine is not.  ta weights layer l-1, tc layer l (Eq. 3: ta = 1 - t, tc = t).
// sin(x) for x in [0, pi]: fold to [0, pi/2] and sum the odd Taylor series through x^11 (the first
// omitted term is below 6e-8 there).  No range reduction, no slow path.
__device__ __forceinline__ float sin_0_pi(float x) {
  const float y = x > 1.57079632679489661923f ? 3.14159265358979323846f - x : x;
  const float y2 = y * y;
  float p = fmaf(y2, -2.50521083854417187751e-8f, 2.75573192239858906526e-6f);  // -1/11!, 1/9!
  p = fmaf(p, y2, -1.98412698412698412698e-4f);                                 // -1/7!
  p = fmaf(p, y2, 8.33333333333333333333e-3f);                                  // 1/5!
  p = fmaf(p, y2, -1.66666666666666666667e-1f);                                 // -1/3!
  return fmaf(p * y2, y, y);
}

// atan2(y, x) for y, x >= 0 (first quadrant), not both zero: z = min / max in [0, 1],
// atan(z) = z P(z^2) with a 9-term polynomial fitted to atan on [0, 1] (maximum error 6e-9 before
// rounding, 1e-7 evaluated in binary32), and atan2 = pi/2 - atan(z) when y > x.
__device__ __forceinline__ float atan2_q1(float y, float x) {
  const float mx = fmaxf(y, x), mn = fminf(y, x);
  const float z = mx > 0.f ? __fdividef(mn, mx) : 0.f;
  const float s = z * z;
  float p = fmaf(s, 2.4567135184e-3f, -1.4401309591e-2f);
  p = fmaf(p, s, 3.9781136401e-2f);
  p = fmaf(p, s, -7.2348490018e-2f);
  p = fmaf(p, s, 1.0498941499e-1f);
  p = fmaf(p, s, -1.4161227780e-1f);
  p = fmaf(p, s, 1.9985906541e-1f);
  p = fmaf(p, s, -3.3332597014e-1f);
  p = fmaf(p, s, 9.9999988638e-1f);
  const float r = z * p;
  return y > x ? 1.57079632679489661923f - r : r;
}

__device__ __forceinline__ RowScalars slerp_scalars(float aa, float cc, float sm, float sp, float ta,
                                                    float tc) {
  RowScalars r;
  // 1/|x| by the hardware reciprocal square root (2 ulp); |x| = |x|^2 / |x|
  const float ra = aa > 0.f ? rsqrtf(aa) : 0.f;
  const float rc = cc > 0.f ? rsqrtf(cc) : 0.f;
  r.na = aa * ra;
  r.nc = cc * rc;
  if (aa > 0.f && cc > 0.f) {
    // h = |u - v| / 2 = sin(Omega / 2), c = |u + v| / 2 = cos(Omega / 2)
    const float h2 = sm > 0.f ? sm * rsqrtf(sm) : 0.f, c2 = sp > 0.f ? sp * rsqrtf(sp) : 0.f;
    const float omega = 2.0f * atan2_q1(h2, c2);
    const float sinw = 0.5f * h2 * c2;  // sin(Omega) = 2 sin(Omega/2) cos(Omega/2)
    r.d = omega * kInvPi;
    if (sinw >= 1e-6f) {
      const float inv = __fdividef(1.0f, sinw);
      r.fa = sin_0_pi(ta * omega) * inv * ra;
      r.fc = sin_0_pi(tc * omega) * inv * rc;
    } else if (sp > sm) {  // same direction: limit of Eq. 3
      r.fa = ta * ra;
      r.fc = tc * rc;
    } else {  // opposite directions: the endpoint t is closer to
      r.fa = tc >= 0.5f ? 0.f : ra;
      r.fc = tc >= 0.5f ? rc : 0.f;
    }
  } else {  // a zero row has no direction: take the other one's
    r.d = 0.f;
    r.fa = ra;
    r.fc = rc;
  }
  return r;
}

#if defined(__CUDACC__)
// Eq. 3's (1 - t, t) for one row: the configured pair, or (MC_T_MAGNITUDE_RATIO) t = |c| / (|a| + |c|)
// from the two squared lengths; 0.5 if both rows are zero.
__device__ __forceinline__ void row_t(int t_mode, float aa, float cc, float& ta, float& tc) {
  if (t_mode == MC_T_MAGNITUDE_RATIO) {
    const float na = aa > 0.f ? aa * rsqrtf(aa) : 0.f, nc = cc > 0.f ? cc * rsqrtf(cc) : 0.f;
    tc = na + nc > 0.f ? __fdividef(nc, na + nc) : 0.5f;
    ta = 1.0f - tc;
  }
}

// One merged row: 16 lanes hold 8 channels each of a (layer l-1) and c (layer l).
template <int DT>
__device__ __forceinline__ void merge_row(const uint4& ra, const uint4& rc, float ta, float tc, int fn, int t_mode, uint4& e_out,
                                          float& g_a, float& g_c, float& d_out) {
  float a[8], c[8];
  {
    const uint32_t wa[4] = {ra.x, ra.y, ra.z, ra.w};
    const uint32_t wc[4] = {rc.x, rc.y, rc.z, rc.w};
#pragma unroll
    for (int i = 0; i < 4; ++i) {
      float2 fa = Elem<DT>::unpack(wa[i]);
      float2 fc = Elem<DT>::unpack(wc[i]);
      a[2 * i] = fa.x;
      a[2 * i + 1] = fa.y;
      c[2 * i] = fc.x;
      c[2 * i + 1] = fc.y;
    }
  }
  float aa = 0.f, cc = 0.f;
#pragma unroll
  for (int i = 0; i < 8; ++i) {
    aa = fmaf(a[i], a[i], aa);
    cc = fmaf(c[i], c[i], cc);
  }
  aa = sum16(aa);
  cc = sum16(cc);
  const float ia = aa > 0.f ? rsqrtf(aa) : 0.f;
  const float ic = cc > 0.f ? rsqrtf(cc) : 0.f;
  // |u - v|^2 and |u + v|^2 formed channel by channel: no cancellation at small or large angles
  float sm = 0.f, sp = 0.f;
#pragma unroll
  for (int i = 0; i < 8; ++i) {
    const float u = a[i] * ia;
    const float dm = fmaf(-c[i], ic, u);
    const float dp = fmaf(c[i], ic, u);
    sm = fmaf(dm, dm, sm);
    sp = fmaf(dp, dp, sp);
  }
  sm = sum16(sm);
  sp = sum16(sp);
  row_t(t_mode, aa, cc, ta, tc);
  RowScalars s = slerp_scalars(aa, cc, sm, sp, ta, tc);
  if (fn != MC_MERGE_SLERP) {  // one vector for both layers: direction of the mean, one magnitude
    float m2 = 0.f;
#pragma unroll
    for (int i = 0; i < 8; ++i) {
      const float h = a[i] + c[i];
      m2 = fmaf(h, h, m2);
    }
    m2 = 0.25f * sum16(m2);
    const float im = m2 > 0.f ? rsqrtf(m2) : 0.f;
    s.fa = s.fc = 0.5f * im;
    s.na = s.nc = fn == MC_MERGE_FMAX ? fmaxf(s.na, s.nc) : m2 * im;
  }
  uint32_t w[4];
  float ee = 0.f;
#pragma unroll
  for (int i = 0; i < 4; ++i) {
    const float x = fmaf(s.fa, a[2 * i], s.fc * c[2 * i]);
    const float y = fmaf(s.fa, a[2 * i + 1], s.fc * c[2 * i + 1]);
    w[i] = Elem<DT>::pack(x, y);
    const float2 r = Elem<DT>::unpack(w[i]);  // the stored value: Eq. 2 divides by its length
    ee = fmaf(r.x, r.x, ee);
    ee = fmaf(r.y, r.y, ee);
  }
  ee = sum16(ee);
  const float il = ee > 0.f ? 1.0f / sqrtf(ee) : 0.f;
  e_out = make_uint4(w[0], w[1], w[2], w[3]);
  g_a = s.na * il;
  g_c = s.nc * il;
  d_out = s.d;
}
#endif

}  // namespace mc
