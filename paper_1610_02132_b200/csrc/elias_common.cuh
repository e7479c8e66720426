// Recursive Elias code (Appendix A.2, Definition A.1) in closed form for integers < 2^16, and
// the MSB-first bit stream the strings S are written to (stream bit t = bit 31 - t % 32 of
// u32 word t / 32).
//
// For k with bit length m the code is P(m) | bin_m(k) | 0, where P(m) is the code of m - 1
// without its final 0: empty for m <= 2, "10"/"11" for m = 3/4, "10" bin_3(m - 1) for
// m = 5..8, "11" bin_4(m - 1) for m = 9..16. Elias(1) is the single bit 0.
#pragma once

#include "qsgd_common.cuh"

namespace qsgd {

__device__ __forceinline__ uint32_t elias_prefix_len(uint32_t m) {
  return (m > 2 ? 2u : 0u) + (m > 4 ? 3u : 0u) + (m > 8 ? 1u : 0u);
}

// |Elias(k)| for 1 <= k < 2^16.
__device__ __forceinline__ uint32_t elias_len(uint32_t k) {
  const uint32_t m = 32u - (uint32_t)__clz((int)k);
  return m == 1 ? 1u : m + 1u + elias_prefix_len(m);
}

// Elias(k), right-aligned in the return value; *len receives its length (<= 23).
__device__ __forceinline__ uint32_t elias_code(uint32_t k, uint32_t* len) {
  const uint32_t m = 32u - (uint32_t)__clz((int)k);
  if (m == 1) { *len = 1; return 0u; }
  uint32_t pv = 0;
  if (m > 8) pv = (3u << 4) | (m - 1u);
  else if (m > 4) pv = (2u << 3) | (m - 1u);
  else if (m > 2) pv = m - 1u;
  *len = m + 1u + elias_prefix_len(m);
  return ((pv << m) | k) << 1;
}

// 32 stream bits starting at absolute bit `pos` (left-aligned in the result).
__device__ __forceinline__ uint32_t peek32(const uint32_t* __restrict__ words, uint64_t pos) {
  const uint64_t idx = pos >> 5;
  const uint32_t w0 = __ldg(words + idx), w1 = __ldg(words + idx + 1);
  return __funnelshift_l(w1, w0, (uint32_t)(pos & 31));
}

// Definition A.1, decoder: N = 1; a leading 1 means "this bit and N more form the new N".
// Reads at most three groups (values < 2^16); returns false on a longer chain.
__device__ __forceinline__ bool elias_read(const uint32_t* __restrict__ words, uint64_t& pos,
                                           uint32_t& value) {
  uint32_t N = 1;
#pragma unroll 1
  for (int it = 0; it < 4; ++it) {
    const uint32_t w = peek32(words, pos);
    if (!(w >> 31)) { pos += 1; value = N; return true; }
    if (it == 3 || N > 15) return false;
    pos += N + 1;
    N = w >> (31 - N);
  }
  return false;
}

// Lane-private writer of a contiguous bit range of the payload. Bits are gathered in a
// left-aligned 64-bit buffer; a word is stored plainly when this writer owns all 32 bits of it
// and OR-ed atomically when it shares the word with a neighbour (payload pre-zeroed).
struct BitWriter {
  uint32_t* words;
  uint64_t widx;     // index of the word the top of `buf` belongs to
  uint64_t buf;      // left-aligned pending bits
  uint32_t nbuf;     // pending bit count (including the lead-in zeros of a shared first word)
  bool first_shared; // the first word starts before this writer's range

  __device__ __forceinline__ void begin(uint32_t* w, uint64_t start_bit) {
    words = w; widx = start_bit >> 5; buf = 0; nbuf = (uint32_t)(start_bit & 31);
    first_shared = nbuf != 0;
  }
  __device__ __forceinline__ void put(uint32_t code, uint32_t len) {   // len in [1, 32]
    buf |= (uint64_t)code << (64 - nbuf - len);
    nbuf += len;
    if (nbuf >= 32) {
      const uint32_t w = (uint32_t)(buf >> 32);
      if (first_shared) { atomicOr(words + widx, w); first_shared = false; }
      else words[widx] = w;
      ++widx; buf <<= 32; nbuf -= 32;
    }
  }
  __device__ __forceinline__ void finish() {
    if (nbuf) atomicOr(words + widx, (uint32_t)(buf >> 32));
  }
};

}  // namespace qsgd
