// LoRA dropout on the branch input of the fine-tuning rows (Section 5: dropout 0.05; the usual
// LoRA placement y = x W + s B A dropout(x)).  The keep decision of element (m, k) - m the row's
// place in the batch's save order, k the input column - is output number c + 1 of the SplitMix64
// stream started at `seed`, c = m * 2^32 + (k >> 2): its 16-bit field k & 3 is compared with
// thr = round(p * 65536).  Forward and backward regenerate the same mask from (seed, m, k); kept
// elements count 1 / (1 - p), applied in fp32 after the contraction so that the bf16 operands
// stay exact copies of the stored values.
#pragma once

#include <stdint.h>

namespace mlora {

struct DropArgs {
  uint64_t seed;
  uint32_t thr;         // 0: dropout off
  float keep_scale;     // 1 / (1 - p)
};

__host__ __device__ __forceinline__ uint64_t drop_bits(uint64_t seed, uint32_t m, uint32_t k4) {
  uint64_t z = seed + ((((uint64_t)m << 32) | (uint64_t)k4) + 1ull) * 0x9E3779B97F4A7C15ull;
  z = (z ^ (z >> 30)) * 0xBF58476D1CE4E5B9ull;
  z = (z ^ (z >> 27)) * 0x94D049BB133111EBull;
  return z ^ (z >> 31);
}
// keep decision of one element
__host__ __device__ __forceinline__ bool drop_keep(const DropArgs& d, uint32_t m, uint32_t k) {
  return (uint32_t)((drop_bits(d.seed, m, k >> 2) >> (16 * (k & 3))) & 0xFFFFu) >= d.thr;
}
// zeroes the dropped ones of four consecutive bf16 held in two 32-bit words (element 0 = low half
// of w0); `z` = drop_bits of their group
__device__ __forceinline__ void drop_mask4(uint64_t z, uint32_t thr, uint32_t& w0, uint32_t& w1) {
  if ((uint32_t)(z & 0xFFFFu) < thr) w0 &= 0xFFFF0000u;
  if ((uint32_t)((z >> 16) & 0xFFFFu) < thr) w0 &= 0x0000FFFFu;
  if ((uint32_t)((z >> 32) & 0xFFFFu) < thr) w1 &= 0xFFFF0000u;
  if ((uint32_t)(z >> 48) < thr) w1 &= 0x0000FFFFu;
}
// eight consecutive bf16 (a 16-byte piece) of row m starting at column k (a multiple of 8)
__device__ __forceinline__ void drop_mask8(const DropArgs& d, uint32_t m, uint32_t k, uint4& v) {
  drop_mask4(drop_bits(d.seed, m, k >> 2), d.thr, v.x, v.y);
  drop_mask4(drop_bits(d.seed, m, (k >> 2) + 1), d.thr, v.z, v.w);
}

}  // namespace mlora
