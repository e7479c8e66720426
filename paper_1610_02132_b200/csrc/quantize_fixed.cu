// Encode, fixed-width path: bucket scale + Philox stochastic rounding + bit packing in one pass
// over the gradient (Section 3.1, Eq. 2; Section 4 bucketing / max-norm; Section 5 bit widths).
//
// One CTA owns a tile of whole buckets (<= 4096 coordinates) staged in shared memory. A thread
// owns groups of 8 consecutive coordinates: it reads them once, contributes a partial sum of
// squares (or maximum) to the bucket reduction, and after the scales are known quantizes the
// same registers, so the gradient is read from HBM exactly once. Sign bits and level fields
// of neighbouring lanes are merged with shuffles into whole 32-bit words before they are
// stored.
#include <float.h>

#include "qsgd_common.cuh"

namespace qsgd {

namespace {

constexpr int kThreads = 256;
constexpr int kTile = 4096;           // coordinates per tile
constexpr int kGroupsPerThread = kTile / 8 / kThreads;  // 2
constexpr int kMaxBucketsPerTile = kTile / 32;          // 128

struct QuantizeParams {
  const float* g;
  uint64_t n;
  uint32_t d;
  uint32_t s;
  uint32_t tile_coords;   // coordinates per tile = whole buckets, <= kTile
  uint32_t k0, k1, step, worker;
  float* A_out;
  uint32_t* sign_out;
  uint32_t* level_out;
  uint64_t B, sign_words, level_words;
};

template <int LB, int NORM>
__global__ void __launch_bounds__(kThreads) quantize_fixed_kernel(const QuantizeParams p) {
  __shared__ __align__(16) float tile[kTile];
  __shared__ float part[kTile / 8];
  __shared__ float s_rcp[kMaxBucketsPerTile];

  const uint32_t tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const uint64_t t0 = (uint64_t)blockIdx.x * p.tile_coords;   // first coordinate of the tile
  const uint64_t left = p.n - t0;
  const uint32_t valid = left < p.tile_coords ? (uint32_t)left : p.tile_coords;

  // ---- stage the tile (coalesced 16-byte loads; zero beyond n) -----------------------------
  for (uint32_t i = tid * 4; i < p.tile_coords; i += kThreads * 4) {
    float4 v = make_float4(0.f, 0.f, 0.f, 0.f);
    if (i + 4 <= valid) {
      v = __ldcs(reinterpret_cast<const float4*>(p.g + t0 + i));
    } else if (i < valid) {
      float t[4] = {0.f, 0.f, 0.f, 0.f};
      for (uint32_t j = 0; i + j < valid; ++j) t[j] = p.g[t0 + i + j];
      v = make_float4(t[0], t[1], t[2], t[3]);
    }
    *reinterpret_cast<float4*>(tile + i) = v;
  }
  __syncthreads();

  // ---- per-group partial of the bucket scale; values stay in registers ---------------------
  float v[kGroupsPerThread][8];
  const uint32_t groups = p.tile_coords >> 3;
#pragma unroll
  for (int j = 0; j < kGroupsPerThread; ++j) {
    const uint32_t grp = tid + j * kThreads;
    float4 a = make_float4(0.f, 0.f, 0.f, 0.f), b = a;
    if (grp < groups) {
      a = *reinterpret_cast<const float4*>(tile + grp * 8);
      b = *reinterpret_cast<const float4*>(tile + grp * 8 + 4);
    }
    v[j][0] = a.x; v[j][1] = a.y; v[j][2] = a.z; v[j][3] = a.w;
    v[j][4] = b.x; v[j][5] = b.y; v[j][6] = b.z; v[j][7] = b.w;
    float acc = 0.f;
#pragma unroll
    for (int e = 0; e < 8; ++e) {
      if (NORM == QSGD_NORM_L2) acc = fmaf(v[j][e], v[j][e], acc);
      else acc = fmaxf(acc, fabsf(v[j][e]));
    }
    if (grp < groups) part[grp] = acc;
  }
  __syncthreads();

  // ---- bucket scales: one warp per bucket, fp64 across the group partials ------------------
  const uint32_t nb = p.tile_coords / p.d;     // buckets in a full tile
  const uint32_t gpb = p.d >> 3;               // groups per bucket
  const uint64_t b0 = t0 / p.d;                // first bucket of the tile
  for (uint32_t b = warp; b < nb; b += kThreads / 32) {
    float A;
    if (NORM == QSGD_NORM_L2) {
      double acc = 0.0;
      for (uint32_t j = lane; j < gpb; j += 32) acc += (double)part[b * gpb + j];
#pragma unroll
      for (int o = 16; o > 0; o >>= 1) acc += __shfl_xor_sync(0xffffffffu, acc, o);
      A = __double2float_rn(__dsqrt_rn(acc));
    } else {
      float acc = 0.f;
      for (uint32_t j = lane; j < gpb; j += 32) acc = fmaxf(acc, part[b * gpb + j]);
#pragma unroll
      for (int o = 16; o > 0; o >>= 1) acc = fmaxf(acc, __shfl_xor_sync(0xffffffffu, acc, o));
      A = acc;
    }
    if (!(A >= FLT_MIN)) A = 0.f;              // zero bucket: Q(0) = 0
    if (lane == 0) {
      s_rcp[b] = A > 0.f ? __frcp_rn(A) : 0.f;
      if (b0 + b < p.B) p.A_out[b0 + b] = A;
    }
  }
  __syncthreads();

  // ---- stochastic rounding and packing -----------------------------------------------------
  const float sf = (float)p.s;
#pragma unroll
  for (int j = 0; j < kGroupsPerThread; ++j) {
    const uint32_t grp = tid + j * kThreads;
    const uint32_t bl = (grp * 8) / p.d;
    const float r = (grp < groups) ? s_rcp[bl] : 0.f;
    const uint64_t i0 = t0 + (uint64_t)grp * 8;       // global index of the group's first value
    const uint64_t q = i0 >> 2;
    const uint4 ra = philox4x32_10((uint32_t)q, (uint32_t)(q >> 32), p.step, p.worker, p.k0, p.k1);
    const uint4 rb = philox4x32_10((uint32_t)(q + 1), (uint32_t)((q + 1) >> 32), p.step, p.worker,
                                   p.k0, p.k1);
    const uint32_t rnd[8] = {ra.x, ra.y, ra.z, ra.w, rb.x, rb.y, rb.z, rb.w};
    uint32_t lv[8];
    uint32_t sb = 0;
#pragma unroll
    for (int e = 0; e < 8; ++e) {
      lv[e] = quantize_level(v[j][e], r, sf, p.s, rnd[e]);
      sb |= (uint32_t)(lv[e] != 0 && v[j][e] < 0.f) << e;
    }
    // sign bitmap: 4 lanes -> one word
    uint32_t sw = sb << (8 * (lane & 3));
    sw |= __shfl_xor_sync(0xffffffffu, sw, 1);
    sw |= __shfl_xor_sync(0xffffffffu, sw, 2);
    const uint64_t sidx = (t0 >> 5) + (grp >> 2);
    if ((lane & 3) == 0 && grp < groups && sidx < p.sign_words) p.sign_out[sidx] = sw;

    if (LB == 8) {
      const uint32_t w0 = lv[0] | lv[1] << 8 | lv[2] << 16 | lv[3] << 24;
      const uint32_t w1 = lv[4] | lv[5] << 8 | lv[6] << 16 | lv[7] << 24;
      const uint64_t widx = (t0 >> 2) + (uint64_t)grp * 2;
      if (grp < groups) {
        if (widx + 1 < p.level_words) *reinterpret_cast<uint2*>(p.level_out + widx) = make_uint2(w0, w1);
        else if (widx < p.level_words) p.level_out[widx] = w0;
      }
    } else if (LB == 4) {
      uint32_t w = 0;
#pragma unroll
      for (int e = 0; e < 8; ++e) w |= lv[e] << (4 * e);
      const uint64_t widx = (t0 >> 3) + grp;
      if (grp < groups && widx < p.level_words) p.level_out[widx] = w;
    } else if (LB == 2) {
      uint32_t w = 0;
#pragma unroll
      for (int e = 0; e < 8; ++e) w |= lv[e] << (2 * e);
      w <<= 16 * (lane & 1);
      w |= __shfl_xor_sync(0xffffffffu, w, 1);
      const uint64_t widx = (t0 >> 4) + (grp >> 1);
      if ((lane & 1) == 0 && grp < groups && widx < p.level_words) p.level_out[widx] = w;
    } else {
      uint32_t w = 0;
#pragma unroll
      for (int e = 0; e < 8; ++e) w |= lv[e] << e;
      w <<= 8 * (lane & 3);
      w |= __shfl_xor_sync(0xffffffffu, w, 1);
      w |= __shfl_xor_sync(0xffffffffu, w, 2);
      const uint64_t widx = (t0 >> 5) + (grp >> 2);
      if ((lane & 3) == 0 && grp < groups && widx < p.level_words) p.level_out[widx] = w;
    }
  }

  // ---- zero the padding of the three regions (last CTA) ------------------------------------
  if (blockIdx.x == gridDim.x - 1 && tid < 4) {
    if (p.B + tid < ((p.B + 3) & ~3ull)) p.A_out[p.B + tid] = 0.f;
    if (p.sign_words + tid < ((p.sign_words + 3) & ~3ull)) p.sign_out[p.sign_words + tid] = 0u;
    if (p.level_words + tid < ((p.level_words + 3) & ~3ull)) p.level_out[p.level_words + tid] = 0u;
  }
}

template <int LB>
int launch_lb(const QuantizeParams& p, int norm_kind, uint32_t grid, cudaStream_t stream) {
  {
    ScopedKernel sk(kKernQuantize, stream);
    if (norm_kind == QSGD_NORM_L2) quantize_fixed_kernel<LB, QSGD_NORM_L2><<<grid, kThreads, 0, stream>>>(p);
    else quantize_fixed_kernel<LB, QSGD_NORM_MAX><<<grid, kThreads, 0, stream>>>(p);
  }
  return (int)cudaGetLastError();
}

}  // namespace

int launch_quantize_fixed(const float* g, uint64_t n, uint32_t d, uint32_t s, int norm_kind,
                          uint64_t seed, uint32_t step, uint32_t worker, uint8_t* out,
                          cudaStream_t stream) {
  const FixedLayout L = make_fixed_layout(n, d, s);
  QuantizeParams p;
  p.g = g; p.n = n; p.d = d; p.s = s;
  p.tile_coords = (kTile / d) * d;
  p.k0 = (uint32_t)seed; p.k1 = (uint32_t)(seed >> 32); p.step = step; p.worker = worker;
  p.A_out = reinterpret_cast<float*>(out);
  p.sign_out = reinterpret_cast<uint32_t*>(out + L.off_sign);
  p.level_out = reinterpret_cast<uint32_t*>(out + L.off_level);
  p.B = L.B; p.sign_words = L.sign_words; p.level_words = L.level_words;
  const uint64_t tiles = (n + p.tile_coords - 1) / p.tile_coords;
  const uint32_t grid = (uint32_t)tiles;
  switch (L.lb) {
    case 1: return launch_lb<1>(p, norm_kind, grid, stream);
    case 2: return launch_lb<2>(p, norm_kind, grid, stream);
    case 4: return launch_lb<4>(p, norm_kind, grid, stream);
    default: return launch_lb<8>(p, norm_kind, grid, stream);
  }
}

}  // namespace qsgd
