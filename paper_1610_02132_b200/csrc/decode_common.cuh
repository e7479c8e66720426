// Reconstruction of +-A * (level / s) from fixed-width fields, shared by the fixed-width decoder
// (fields read from the message) and the Elias decoder (fields rebuilt in shared memory).
#pragma once

#include "qsgd_common.cuh"

namespace qsgd {

__device__ __forceinline__ float shfl_f(float v, uint32_t src) {
  return __shfl_sync(0xffffffffu, v, (int)src);
}

// Adds peer k's 16 values to acc[]. SINGLE: the whole chunk lies in one bucket and `lut` is
// already scaled by A; otherwise `lut` holds +-(level / s) and A is this lane's bucket scale.
template <int LB, bool SINGLE>
__device__ __forceinline__ void add_peer_lut(float (&acc)[16], const uint32_t (&w)[4], uint32_t sb,
                                             float lut, float A) {
  if (LB == 4) {
#pragma unroll
    for (int h = 0; h < 2; ++h) {
      const uint32_t word = w[h], s8 = sb >> (8 * h);
      const uint32_t ev = word & 0x0F0F0F0Fu, od = (word >> 4) & 0x0F0F0F0Fu;
      const uint32_t ie = (((s8 & 0x55u) * 0x00410410u) & 0x10101010u) | ev;   // coords 0,2,4,6
      const uint32_t io = (((s8 & 0xAAu) * 0x00208208u) & 0x10101010u) | od;   // coords 1,3,5,7
#pragma unroll
      for (int j = 0; j < 4; ++j) {
        float a = shfl_f(lut, ie >> (8 * j));
        float b = shfl_f(lut, io >> (8 * j));
        if (!SINGLE) { a = __fmul_rn(A, a); b = __fmul_rn(A, b); }
        acc[8 * h + 2 * j] = __fadd_rn(acc[8 * h + 2 * j], a);
        acc[8 * h + 2 * j + 1] = __fadd_rn(acc[8 * h + 2 * j + 1], b);
      }
    }
  } else if (LB == 2) {
    // 16 two-bit levels in w[0]. Per half (8 coordinates) spread the levels to nibble spacing
    // and drop the sign bit at bit 2 of each nibble; the lookup table repeats every 8 lanes, so
    // whatever follows in the shifted word is ignored by the shuffle (it reads 5 index bits).
#pragma unroll
    for (int h = 0; h < 2; ++h) {
      uint32_t x = (w[0] >> (16 * h)) & 0xFFFFu;
      x = (x | (x << 8)) & 0x00FF00FFu;
      x = (x | (x << 4)) & 0x0F0F0F0Fu;
      x = (x | (x << 2)) & 0x33333333u;
      uint32_t y = (sb >> (8 * h)) & 0xFFu;
      y = (y | (y << 12)) & 0x000F000Fu;
      y = (y | (y << 6)) & 0x03030303u;
      y = (y | (y << 3)) & 0x11111111u;
      const uint32_t z = x | (y << 2);
#pragma unroll
      for (int j = 0; j < 8; ++j) {
        float a = shfl_f(lut, z >> (4 * j));
        if (!SINGLE) a = __fmul_rn(A, a);
        acc[8 * h + j] = __fadd_rn(acc[8 * h + j], a);
      }
    }
  } else {
    // LB = 1: interleave the 16 level bits (even positions) with the 16 sign bits (odd); the
    // lookup table repeats every 4 lanes.
    uint32_t x = w[0] & 0xFFFFu, y = sb & 0xFFFFu;
    x = (x | (x << 8)) & 0x00FF00FFu; y = (y | (y << 8)) & 0x00FF00FFu;
    x = (x | (x << 4)) & 0x0F0F0F0Fu; y = (y | (y << 4)) & 0x0F0F0F0Fu;
    x = (x | (x << 2)) & 0x33333333u; y = (y | (y << 2)) & 0x33333333u;
    x = (x | (x << 1)) & 0x55555555u; y = (y | (y << 1)) & 0x55555555u;
    const uint32_t z = x | (y << 1);
#pragma unroll
    for (int e = 0; e < 16; ++e) {
      float a = shfl_f(lut, z >> (2 * e));
      if (!SINGLE) a = __fmul_rn(A, a);
      acc[e] = __fadd_rn(acc[e], a);
    }
  }
}

// LB = 8: table lookup of level / s in shared memory (entry l of lane t at word l * 32 + t).
__device__ __forceinline__ void add_peer_tab(float (&acc)[16], const uint32_t (&w)[4], uint32_t sb,
                                             const uint8_t* tab_lane, float A) {
#pragma unroll
  for (int h = 0; h < 4; ++h) {
#pragma unroll
    for (int j = 0; j < 4; ++j) {
      const uint32_t off = (j == 0 ? (w[h] << 7) : (w[h] >> (8 * j - 7))) & 0x7F80u;
      const float xi = *reinterpret_cast<const float*>(tab_lane + off);
      const uint32_t m = __float_as_uint(__fmul_rn(A, xi)) ^ ((sb << (31 - (4 * h + j))) & 0x80000000u);
      acc[4 * h + j] = __fadd_rn(acc[4 * h + j], __uint_as_float(m));
    }
  }
}


// Writes 16 accumulated values of one lane: acc as it is, or the SGD step x <- x - c * acc.
template <bool FUSED>
__device__ __forceinline__ void store_lane16(float* o, const float (&acc)[16], uint64_t i0, uint64_t n,
                                             float c) {
  if (i0 + 16 <= n) {
#pragma unroll
    for (int j = 0; j < 4; ++j) {
      float4 r = make_float4(acc[4 * j], acc[4 * j + 1], acc[4 * j + 2], acc[4 * j + 3]);
      if (FUSED) {
        const float4 x = *reinterpret_cast<const float4*>(o + 4 * j);
        r.x = __fsub_rn(x.x, __fmul_rn(c, r.x)); r.y = __fsub_rn(x.y, __fmul_rn(c, r.y));
        r.z = __fsub_rn(x.z, __fmul_rn(c, r.z)); r.w = __fsub_rn(x.w, __fmul_rn(c, r.w));
      }
      *reinterpret_cast<float4*>(o + 4 * j) = r;
    }
  } else {
#pragma unroll
    for (int e = 0; e < 16; ++e)
      if (i0 + e < n) o[e] = FUSED ? __fsub_rn(o[e], __fmul_rn(c, acc[e])) : acc[e];
  }
}

// Where `want` consecutive coordinates of bucket b, starting at bucket-relative position c0, live in
// the output array, and how many of them exist.
struct OutSpan {
  float* ptr;
  uint32_t valid;
};

__device__ __forceinline__ OutSpan out_span(float* out, const BucketMap& map, uint64_t b, uint32_t c0, uint32_t d,
                                            uint64_t n, uint32_t want) {
  OutSpan sp;
  if (map.src) {
    const uint32_t L = __ldg(map.len + b);
    sp.ptr = out + __ldg(map.src + b) + c0;
    sp.valid = c0 < L ? min(want, L - c0) : 0u;
  } else {
    const uint64_t i0 = b * d + c0;
    sp.ptr = out + i0;
    sp.valid = i0 < n ? (uint32_t)min((uint64_t)want, n - i0) : 0u;
  }
  return sp;
}

// store_lane16 through a span: vector accesses when all 16 values exist and the place is 16-byte
// aligned, element by element otherwise.
template <bool FUSED>
__device__ __forceinline__ void store_span16(const OutSpan& sp, const float (&acc)[16], float c) {
  if (sp.valid == 16u && (reinterpret_cast<uintptr_t>(sp.ptr) & 15u) == 0) {
    store_lane16<FUSED>(sp.ptr, acc, 0, 16, c);
  } else {
#pragma unroll
    for (int e = 0; e < 16; ++e)
      if ((uint32_t)e < sp.valid) sp.ptr[e] = FUSED ? __fsub_rn(sp.ptr[e], __fmul_rn(c, acc[e])) : acc[e];
  }
}

}  // namespace qsgd
