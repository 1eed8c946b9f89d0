// The 4-bit shared cache (Sec. 5: MiniCache on top of 4-bit KIVI quantisation): tile geometry and the
// device-side pieces every kernel that reads it shares.  The byte layout is described at
// mc_pair_cache in minicache.h.
#pragma once
#include "mc_common.cuh"

namespace mc {

constexpr int kQ4Page = 32;                    // tokens per page = quantisation group of the keys
constexpr int kQ4CodeBytes = kQ4Page * 64;     // 2048: 32 rows of 128 four-bit codes
constexpr int kQ4GroupBytes = 512;             // group parameters (scales, zeros) of a tile
constexpr int kQ4ScaleOff = kQ4CodeBytes + kQ4GroupBytes;       // the two layers' fp32 scales [2][32]
constexpr int kQ4TileBytes = kQ4ScaleOff + 2 * kQ4Page * 4;     // 2816
constexpr int kResTileBytes = kQ4Page * kRowBytes + 2 * kQ4Page * 4;  // a 16-bit tile of 32 tokens: 8448

#if defined(__CUDACC__)
// Four pairs of codes out of one 32-bit word as exact small integers of the 16-bit type: pair n holds
// the nibbles at bits [4n, 4n+4) and [16 + 4n, 16 + 4n + 4).  The nibble is OR-ed into the mantissa of
// a constant whose unit in the last place matches the nibble's position, and the constant is
// subtracted again (exact): no integer-to-float conversion instruction is involved.
template <int DT>
__device__ __forceinline__ void code_pairs(uint32_t w, uint32_t (&c)[4]);
template <>
__device__ __forceinline__ void code_pairs<MC_F16>(uint32_t w, uint32_t (&c)[4]) {
  // binary16: bits 0..3 of the mantissa count units at 1024, bits 4..7 count units at 64
  const uint32_t w8 = w >> 8;
  uint32_t r[4] = {(w & 0x000F000Fu) | 0x64006400u, (w & 0x00F000F0u) | 0x54005400u, (w8 & 0x000F000Fu) | 0x64006400u,
                   (w8 & 0x00F000F0u) | 0x54005400u};
  const __half2 k1024 = __half2half2(__ushort_as_half((unsigned short)0x6400));
  const __half2 k64 = __half2half2(__ushort_as_half((unsigned short)0x5400));
#pragma unroll
  for (int n = 0; n < 4; ++n) {
    const __half2 v = __hsub2(*reinterpret_cast<__half2*>(&r[n]), (n & 1) ? k64 : k1024);
    c[n] = *reinterpret_cast<const uint32_t*>(&v);
  }
}
template <>
__device__ __forceinline__ void code_pairs<MC_BF16>(uint32_t w, uint32_t (&c)[4]) {
  // bfloat16 has seven mantissa bits: only bits 0..3 can take a nibble (units at 128)
  const __nv_bfloat162 k128 = __bfloat162bfloat162(__ushort_as_bfloat16((unsigned short)0x4300));
#pragma unroll
  for (int n = 0; n < 4; ++n) {
    uint32_t r = ((w >> (4 * n)) & 0x000F000Fu) | 0x43004300u;
    const __nv_bfloat162 v = __hsub2(*reinterpret_cast<__nv_bfloat162*>(&r), k128);
    c[n] = *reinterpret_cast<const uint32_t*>(&v);
  }
}

// code * scale + zero on a pair of elements, rounded once to the 16-bit type: the stored direction of
// the 4-bit cache, and directly a tensor-core operand register.
template <int DT>
__device__ __forceinline__ uint32_t deq_pair(uint32_t code, uint32_t scale, uint32_t zero) {
  if (DT == MC_F16) {
    const __half2 v = __hfma2(*reinterpret_cast<__half2*>(&code), *reinterpret_cast<__half2*>(&scale),
                              *reinterpret_cast<__half2*>(&zero));
    return *reinterpret_cast<const uint32_t*>(&v);
  } else {
    const __nv_bfloat162 v = __hfma2(*reinterpret_cast<__nv_bfloat162*>(&code), *reinterpret_cast<__nv_bfloat162*>(&scale),
                                     *reinterpret_cast<__nv_bfloat162*>(&zero));
    return *reinterpret_cast<const uint32_t*>(&v);
  }
}

// Chunk position of the group parameters of the channels [8 o, 8 o + 8) in a K tile, and of chunk c of
// token-pair block i in a V tile.
__host__ __device__ __forceinline__ int q4_kmeta_pos(int o) { return 4 * (o & 3) + (o >> 2); }
__host__ __device__ __forceinline__ int q4_vchunk_pos(int i, int c) { return c ^ ((i & 3) << 1); }
// Channel of nibble n (0..3) of word k (0..3) of chunk c (0..7) of a V token-pair block.
__host__ __device__ __forceinline__ int q4_vchannel(int c, int k, int n) { return 32 * k + 16 * (n >> 1) + 8 * (n & 1) + c; }
#endif

}  // namespace mc
