// Dropout masks from a counter-based generator, shared by the element-wise kernels and the attention kernels.
// Philox4x32-10 (Salmon, Moraes, Dror, Shaw, "Parallel random numbers: as easy as 1, 2, 3", SC'11): key = the 64-bit
// seed, counter = (element / 4 as two words, site, step); element e takes word e % 4 of the block and is kept iff the
// word >= thr = floor(p 2^32); kept values are multiplied by scale = 1 / (1 - p).  thr = 0 switches a site off.
#pragma once
#include <cuda_runtime.h>
#include <stdint.h>

namespace hift {

struct DropArgs { uint32_t k0, k1, site, step, thr; float scale; };

__device__ __forceinline__ uint4 philox4x32_10(uint4 c, uint32_t k0, uint32_t k1) {
#pragma unroll
  for (int r = 0; r < 10; ++r) {
    const uint32_t hi0 = __umulhi(0xD2511F53u, c.x), lo0 = 0xD2511F53u * c.x;
    const uint32_t hi1 = __umulhi(0xCD9E8D57u, c.z), lo1 = 0xCD9E8D57u * c.z;
    c = make_uint4(hi1 ^ c.y ^ k0, lo1, hi0 ^ c.w ^ k1, lo0);
    k0 += 0x9E3779B9u;
    k1 += 0xBB67AE85u;
  }
  return c;
}

// Attention probabilities (site 1000 + block): element ((b H + h) S + q) S' + k with S' = S rounded up to a multiple of 4,
// so that one generator block holds keys k4 .. k4 + 3 (k4 a multiple of 4) of one query row.  `bh` = b H + h.
__device__ __forceinline__ uint4 attn_drop_words(const DropArgs& a, int bh, int S, int q, int k4) {
  const size_t sp = (size_t)((S + 3) & ~3);
  const size_t blk = (((size_t)bh * (size_t)S + (size_t)q) * sp + (size_t)k4) >> 2;
  return philox4x32_10(make_uint4((uint32_t)blk, (uint32_t)(blk >> 32), a.site, a.step), a.k0, a.k1);
}
__device__ __forceinline__ uint32_t word_of(const uint4& w, int i) { return i == 0 ? w.x : i == 1 ? w.y : i == 2 ? w.z : w.w; }

}  // namespace hift
