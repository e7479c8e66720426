// Encode, fixed-width path: bucket scale + Philox stochastic rounding + bit packing in one pass
// over the gradient (Section 3.1, Eq. 2; Section 4 bucketing / max-norm; Section 5 bit widths).
//
// Three streaming kernels for power-of-two bucket sizes, all persistent and fed by 1-D TMA bulk
// copies (cp.async.bulk + mbarrier), so no thread spends instructions on global loads:
//   * quantize_warp_kernel (d <= 512, with or without a bucket map): every warp runs its own pipeline over
//     chunks of 512 coordinates (whole buckets) with a private ring of shared-memory stages that
//     its lane 0 refills as soon as the warp has taken a stage into registers. No CTA-wide
//     barrier and no separate "empty" barrier exist, and every decision is warp-uniform.
//   * quantize_group_kernel (d >= 1024, 2-norm, no bucket map): the same per-warp pipelines; the
//     warps that share a bucket meet once per chunk at a named barrier of their own to exchange
//     their partial sums.
//   * quantize_pow2_kernel (d >= 1024, max-norm or bucket map, where it measures faster): the CTA
//     walks tiles of 4096 coordinates through a shared ring; scales of buckets that span several
//     warps meet in shared memory.
// A thread owns 16 consecutive coordinates: it pulls them into registers once, the bucket scale
// is reduced with shuffles, and the same registers are then quantized, so the gradient is read
// from HBM exactly once. The kernels are bound by the integer (ALU) and multiply (FMA-heavy)
// pipes, which Philox alone loads with 2 + 2 instructions per round; everything else is written
// to stay off those two pipes where it can:
//   * the uniform u = m * 2^-24 (m = top 24 Philox bits) needs no integer-to-float conversion:
//     the bit pattern m read as an fp32 is the subnormal (or smallest-normal) number m * 2^-149,
//     and fma(that, 2^125, t) has the exact product m * 2^-24 and rounds once, exactly like
//     t + u (subnormal operands are not flushed: the library is compiled without -ftz);
//   * with the 2-norm, a level can exceed s only at a coordinate that holds nearly all of its
//     bucket's norm; a warp checks that once per chunk and skips the per-coordinate clamp
//     otherwise;
//   * floor(c) is the round-down add c + 2^23, whose mantissa then holds the integer;
//   * level fields are packed by Horner multiply-adds on those raw float bits, the constant
//     exponent bits being removed once per word;
//   * the sign bit "negative and level > 0" is the sign of fma(level, v, +0), shifted into the
//     sign word with a funnel shift.
// A generic kernel (any bucket size that is a multiple of 32) keeps the simple structure.
#include <float.h>

#include <atomic>

#include "qsgd_common.cuh"

namespace qsgd {

namespace {

constexpr int kThreads = 256;
constexpr int kTile = 4096;           // coordinates per tile

struct QuantizeParams {
  const float* g;
  uint64_t n;
  uint32_t d;
  uint32_t s;
  uint32_t tile_coords;   // generic kernel: coordinates per tile = whole buckets, <= kTile
  uint64_t coord_base;    // generic kernel: first coordinate it is responsible for
  uint32_t k0, k1, step, worker;
  float* A_out;
  uint32_t* sign_out;
  uint32_t* level_out;
  uint64_t B, sign_words, level_words;
  uint64_t tiles;
  uint32_t* status;
  uint64_t* info;         // optional: the four message-info words of a fixed-width message
  uint64_t total_bytes;
  uint32_t* clear_word;   // optional: a word the kernel sets to zero (arrival counter of a later kernel)
  BucketMap map;          // per-tensor policy: where each bucket lives in g, or no map
};

// ---------------------------------------------------------------------------------------------
// PTX helpers: mbarrier and 1-D bulk copy global -> shared.
// ---------------------------------------------------------------------------------------------
__device__ __forceinline__ uint32_t smem_u32(const void* p) {
  return (uint32_t)__cvta_generic_to_shared(p);
}
__device__ __forceinline__ void mbar_init(uint64_t* bar, uint32_t count) {
  asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(smem_u32(bar)), "r"(count) : "memory");
}
__device__ __forceinline__ void mbar_expect_tx(uint64_t* bar, uint32_t bytes) {
  asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(smem_u32(bar)), "r"(bytes)
               : "memory");
}
__device__ __forceinline__ void bulk_load(void* dst, const void* src, uint32_t bytes, uint64_t* bar) {
  asm volatile(
      "cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];" ::"r"(
          smem_u32(dst)),
      "l"(src), "r"(bytes), "r"(smem_u32(bar))
      : "memory");
}
__device__ __forceinline__ bool mbar_try_wait(uint64_t* bar, uint32_t parity) {
  uint32_t ok;
  asm volatile(
      "{\n\t.reg .pred p;\n\t"
      "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\t"
      "selp.u32 %0, 1, 0, p;\n\t}"
      : "=r"(ok)
      : "r"(smem_u32(bar)), "r"(parity)
      : "memory");
  return ok != 0;
}
// Bounded wait: gives up after `polls` tries and reports it instead of spinning forever.
constexpr uint32_t kDrainPolls = 1u << 22;   // bound of the waits that drain copies in flight
__device__ __forceinline__ bool mbar_wait_bounded(uint64_t* bar, uint32_t parity, uint32_t polls) {
  for (uint32_t it = 0; it < polls; ++it)
    if (mbar_try_wait(bar, parity)) return true;
  return false;
}
__device__ __forceinline__ void mbar_arrive(uint64_t* bar) {
  asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(smem_u32(bar)) : "memory");
}
__device__ __forceinline__ float fma_rn(float a, float b, float c) {
  float r;
  asm("fma.rn.f32 %0, %1, %2, %3;" : "=f"(r) : "f"(a), "f"(b), "f"(c));
  return r;
}

// ---------------------------------------------------------------------------------------------
// Philox4x32-10 for the counter (q, 0, step, worker) with everything that does not depend on q
// folded into kernel-uniform constants on the host: after round 0 two of the four words are
// constants, which also makes one product of round 1 a constant. 37 instead of 40
// multiply / xor instructions per block of four uniforms.
// ---------------------------------------------------------------------------------------------
struct PhiloxConsts {
  uint32_t y0;        // worker ^ k1[0]
  uint32_t z0;        // lo(M1 * step) ^ k0[1]
  uint32_t z1;        // hi(M0 * x0) ^ k1[1],  x0 = hi(M1 * step) ^ k0[0]
  uint32_t z2;        // lo(M0 * x0) ^ k1[2]
  uint32_t k0_2;      // k0[2]
  uint32_t k[7][2];   // round keys 3 .. 9
};

constexpr uint32_t kM0 = 0xD2511F53u, kM1 = 0xCD9E8D57u;

__device__ __forceinline__ uint4 philox_q(uint32_t q, const PhiloxConsts& pc) {
  // round 0: (q, 0, step, worker) -> (x0, l1, hi(M0 q) ^ y0, lo(M0 q))
  uint64_t p0 = (uint64_t)kM0 * q;
  uint32_t a2 = (uint32_t)(p0 >> 32) ^ pc.y0, a3 = (uint32_t)p0;
  // round 1: (x0, l1, a2, a3) -> (hi(M1 a2) ^ z0, lo(M1 a2), a3 ^ z1, lo(M0 x0))
  uint64_t p1 = (uint64_t)kM1 * a2;
  uint32_t c0 = (uint32_t)(p1 >> 32) ^ pc.z0, c1 = (uint32_t)p1, c2 = a3 ^ pc.z1;
  // round 2: c3 = lo(M0 x0) is folded into z2
  p0 = (uint64_t)kM0 * c0;
  p1 = (uint64_t)kM1 * c2;
  c0 = (uint32_t)(p1 >> 32) ^ c1 ^ pc.k0_2;
  c1 = (uint32_t)p1;
  c2 = (uint32_t)(p0 >> 32) ^ pc.z2;
  uint32_t c3 = (uint32_t)p0;
  // rounds 3 .. 9: the high and low halves by separate multiplies (measured slightly faster than the
  // 64-bit products here; the first rounds stay as they are, where it measured slower)
#pragma unroll
  for (int r = 0; r < 7; ++r) {
    const uint32_t h0 = __umulhi(kM0, c0), l0 = kM0 * c0;
    const uint32_t h1 = __umulhi(kM1, c2), l1 = kM1 * c2;
    c0 = h1 ^ c1 ^ pc.k[r][0];
    c1 = l1;
    c2 = h0 ^ c3 ^ pc.k[r][1];
    c3 = l0;
  }
  return make_uint4(c0, c1, c2, c3);
}

// The uniforms of the 16 coordinates of one thread (Philox blocks q0 .. q0 + 3) as fp32 bit
// patterns m = word >> 8 (see quantize_one).
__device__ __forceinline__ void philox_uniforms16(uint32_t q0, const PhiloxConsts& pc, float (&um)[16]) {
#pragma unroll
  for (int b = 0; b < 4; ++b) {
    const uint4 w = philox_q(q0 + b, pc);
    um[4 * b] = __uint_as_float(w.x >> 8);
    um[4 * b + 1] = __uint_as_float(w.y >> 8);
    um[4 * b + 2] = __uint_as_float(w.z >> 8);
    um[4 * b + 3] = __uint_as_float(w.w >> 8);
  }
}

constexpr float kTwo23 = 8388608.0f;
constexpr uint32_t kTwo23Bits = 0x4B000000u;

constexpr float kTwo125 = 4.253529586511730793292182592897102643e+37f;

// One coordinate. Returns the raw bits of 2^23 + level (level clamped to s when CLAMP); pushes the
// sign bit into `sw`. `um` is the bit pattern m = top 24 Philox bits read as an fp32, i.e. m * 2^-149.
// RAW_SIGN: push the sign bit of v as it is; the caller clears the signs of zero levels afterwards
// with a mask derived from the packed level words (cheaper than two more operations per coordinate
// when a word holds many fields).
template <bool RAW_SIGN, bool CLAMP>
__device__ __forceinline__ uint32_t quantize_one(float v, float r, float sf, float cap, float um,
                                                 uint32_t& sw) {
  const float t = __fmul_rn(__fmul_rn(sf, fabsf(v)), r);
  const float c = fma_rn(um, kTwo125, t);                    // t + m * 2^-24, one rounding
  float fl = __fadd_rd(c, kTwo23);                           // 2^23 + floor(c)
  if (CLAMP) fl = fminf(fl, cap);                            // 2^23 + min(floor(c), s)
  if (RAW_SIGN) {
    sw = __funnelshift_l(__float_as_uint(v), sw, 1);
  } else {
    const float lf = __fsub_rn(fl, kTwo23);                 // the level as a float, exact
    const float sv = fma_rn(lf, v, 0.0f);                   // sign set iff level > 0 and v < 0
    sw = __funnelshift_l(__float_as_uint(sv), sw, 1);
  }
  return __float_as_uint(fl);
}

// Rounds and packs the 16 coordinates of a thread, highest first: level fields by Horner
// multiply-adds on the raw float bits (the constant exponent bits are removed once per word),
// sign bits by funnel shifts; signs of zero levels are cleared at the end.
template <int LB, bool CLAMP>
__device__ __forceinline__ void quantize16(const float (&v)[16], const float (&um)[16], float r, float sf,
                                           float cap, uint32_t (&lw)[4], uint32_t& sw) {
  sw = 0;
#pragma unroll
  for (int j = 0; j < 4; ++j) lw[j] = 0u;                 // LB = 8: 4 words; 4: 2; 2: 1; 1: half
#pragma unroll
  for (int c4 = 3; c4 >= 0; --c4) {
#pragma unroll
    for (int e = 3; e >= 0; --e) {
      const uint32_t bits = quantize_one<LB != 8, CLAMP>(v[4 * c4 + e], r, sf, cap, um[4 * c4 + e], sw);
      if (LB == 8) lw[c4] = lw[c4] * 256u + bits;
      else if (LB == 4) lw[c4 >> 1] = lw[c4 >> 1] * 16u + bits;
      else if (LB == 2) lw[0] = lw[0] * 4u + bits;
      else lw[0] = lw[0] * 2u + bits;
    }
  }
  // remove the exponent bits that rode along: sum over the fields of 0x4B000000 << (LB * e)
  if (LB == 8) {
#pragma unroll
    for (int j = 0; j < 4; ++j) lw[j] -= kTwo23Bits * 0x01010101u;
  } else if (LB == 4) {
    lw[0] -= kTwo23Bits * 0x11111111u;
    lw[1] -= kTwo23Bits * 0x11111111u;
  } else if (LB == 2) {
    lw[0] -= kTwo23Bits * 0x55555555u;
  } else {
    lw[0] = (lw[0] - kTwo23Bits * 0xFFFFu) & 0xFFFFu;
  }
}

// Bit e of the result is set iff level field e of the 16 coordinates packed in lw is nonzero.
template <int LB>
__device__ __forceinline__ uint32_t nonzero_fields16(const uint32_t (&lw)[4]) {
  if (LB == 1) return lw[0] & 0xFFFFu;
  if (LB == 2) {
    uint32_t y = (lw[0] | (lw[0] >> 1)) & 0x55555555u;
    y = (y | (y >> 1)) & 0x33333333u;
    y = (y | (y >> 2)) & 0x0F0F0F0Fu;
    y = (y | (y >> 4)) & 0x00FF00FFu;
    return (y | (y >> 8)) & 0xFFFFu;
  }
  uint32_t m = 0;                                           // LB == 4: two words of eight fields
#pragma unroll
  for (int h = 0; h < 2; ++h) {
    uint32_t y = lw[h] | (lw[h] >> 1);
    y = (y | (y >> 2)) & 0x11111111u;
    y = (y | (y >> 3)) & 0x03030303u;
    y = (y | (y >> 6)) & 0x000F000Fu;
    m |= ((y | (y >> 12)) & 0xFFu) << (8 * h);
  }
  return m;
}

// Stores the sign and level words of the 16 coordinates of every lane of a warp; `c` is the index
// of the warp's chunk of 512 coordinates (complete chunks only: no bounds to check).
template <int LB>
__device__ __forceinline__ void store_chunk(uint32_t* sign_out, uint32_t* level_out, uint32_t c, uint32_t lane,
                                            uint32_t sw, const uint32_t (&lw)[4]) {
  {
    uint32_t w = (sw & 0xFFFFu) << (16 * (lane & 1));
    w |= __shfl_xor_sync(0xffffffffu, w, 1);
    if ((lane & 1) == 0) sign_out[c * 16u + (lane >> 1)] = w;
  }
  if (LB == 8) {
    *reinterpret_cast<uint4*>(level_out + ((size_t)c * 128u + lane * 4u)) = make_uint4(lw[0], lw[1], lw[2], lw[3]);
  } else if (LB == 4) {
    *reinterpret_cast<uint2*>(level_out + ((size_t)c * 64u + lane * 2u)) = make_uint2(lw[0], lw[1]);
  } else if (LB == 2) {
    level_out[(size_t)c * 32u + lane] = lw[0];
  } else {
    uint32_t w = lw[0] << (16 * (lane & 1));
    w |= __shfl_xor_sync(0xffffffffu, w, 1);
    if ((lane & 1) == 0) level_out[c * 16u + (lane >> 1)] = w;
  }
}

constexpr int kStages = 3;

struct __align__(16) TileSmem {
  float tile[kStages][kTile];
  float wsum[2][kThreads / 32];
  double wsum64[kThreads / 32];
  uint64_t full[kStages];    // bulk copy landed
  uint64_t empty[kStages];   // all warps have taken their values out of the stage
};

struct FastParams {
  const float* g;
  uint32_t full_tiles;      // tiles of 4096 coordinates, all complete
  uint32_t log2d;           // bucket size 2^log2d, 5 .. 12
  uint32_t s;
  float* A_out;
  uint32_t* sign_out;
  uint32_t* level_out;
  uint32_t* status;
  uint64_t* info;           // optional message-info words, written by CTA 0
  uint64_t total_bytes;
  uint32_t* clear_word;     // optional word set to zero by CTA 0
  PhiloxConsts pc;
  uint32_t main_ctas;       // CTAs that stream complete tiles
  uint32_t poll_limit;      // bound of the main-loop waits (the final drain keeps its own bound)
  BucketMap map;            // per-tensor policy: where each bucket lives in g (quads set), or no map
  QuantizeParams tail;      // parameters of the extra CTA (used when gridDim.x > main_ctas)
};

template <int LB, int NORM, bool MAPPED>
__device__ __forceinline__ void quantize_generic_tile(const QuantizeParams& p, uint32_t block, uint32_t nblocks,
                                                      float* tile, float* part, float* s_rcp);

// Producer side of one stage, called by all lanes of warp 0: start the bulk copies of tile t.
// Ordinary case: lane 0 starts one copy of the whole tile. With a bucket map, lane j looks up
// bucket j of the tile (at most 16 buckets: d >= 256); when the buckets are complete and follow one
// another in memory (the rule inside a tensor) it is again one copy, otherwise every lane copies its
// own bucket and puts zeros behind a short one (plain stores, made visible to the consumers by the
// warp barrier before lane 0's expect-tx arrive, which releases). The map guarantees 16-byte aligned
// places and lengths.
template <bool MAPPED>
__device__ __forceinline__ void issue_tile(const FastParams& p, float* tile, uint64_t* full_bar, uint32_t t,
                                           uint32_t lane) {
  if (!MAPPED) {
    if (lane == 0) {
      mbar_expect_tx(full_bar, kTile * 4);
      bulk_load(tile, p.g + (size_t)t * kTile, kTile * 4, full_bar);
    }
    return;
  }
  const uint32_t d = 1u << p.log2d, nb = kTile >> p.log2d;
  const uint64_t b0 = (uint64_t)t << (12u - p.log2d);
  uint32_t L = 0;
  uint64_t src = 0;
  if (lane < nb) {
    L = min(__ldg(p.map.len + b0 + lane), d);
    src = __ldg(p.map.src + b0 + lane);
  }
  const uint64_t src0 = __shfl_sync(0xffffffffu, src, 0);
  const bool in_line = lane >= nb || (L == d && src == src0 + (uint64_t)lane * d);
  if (__all_sync(0xffffffffu, in_line)) {
    if (lane == 0) {
      mbar_expect_tx(full_bar, kTile * 4);
      bulk_load(tile, p.g + src0, kTile * 4, full_bar);
    }
    return;
  }
  if (lane < nb)
    for (uint32_t c = L; c < d; c += 4) *reinterpret_cast<float4*>(tile + lane * d + c) = make_float4(0.f, 0.f, 0.f, 0.f);
  uint32_t bytes = lane < nb ? 4u * L : 0u;
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) bytes += __shfl_xor_sync(0xffffffffu, bytes, o);
  __syncwarp();
  if (lane == 0) mbar_expect_tx(full_bar, bytes);
  __syncwarp();
  if (lane < nb && L) bulk_load(tile + lane * d, p.g + src, 4u * L, full_bar);
}

// CTA-wide streaming kernel for d >= 1024, where a bucket spans 2^(log2d - 9) warps and the scales
// meet in shared memory. CTAs 0 .. main_ctas - 1 stream the complete tiles; one optional extra CTA
// runs the ragged last tile and the region padding through the generic tile code (its operands alias
// the tile ring). MAPPED: buckets are fetched through a bucket map (per-tensor policy); a separate
// instantiation, so that the ordinary kernel carries none of that code.
template <int LB, int NORM, bool MAPPED>
__global__ void __launch_bounds__(kThreads, 4)
quantize_pow2_kernel(const __grid_constant__ FastParams p) {
  extern __shared__ __align__(128) uint8_t smem_raw[];
  TileSmem& sm = *reinterpret_cast<TileSmem*>(smem_raw);

  const uint32_t tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const uint32_t grid = p.main_ctas;
  if (blockIdx.x >= grid) {                     // the extra CTA: ragged tail + padding
    chain_wait();
    quantize_generic_tile<LB, NORM, MAPPED>(p.tail, 0u, 1u, sm.tile[0], sm.tile[1], sm.tile[1] + 1024);
    return;
  }
  if (tid == 0) {
    for (int s = 0; s < kStages; ++s) {
      mbar_init(&sm.full[s], 1);
      mbar_init(&sm.empty[s], kThreads / 32);
    }
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  chain_wait();                                 // nothing above touches global memory
  __syncthreads();
  if (MAPPED ? warp == 0 : tid == 0) {
    if (tid == 0 && blockIdx.x == 0 && p.info) {
      p.info[0] = 8 * p.total_bytes; p.info[1] = 0; p.info[2] = p.total_bytes; p.info[3] = 0;
    }
    if (tid == 0 && blockIdx.x == 0 && p.clear_word) *p.clear_word = 0u;
    for (int s = 0; s < kStages; ++s) {
      const uint32_t t = blockIdx.x + (uint32_t)s * grid;
      if (t < p.full_tiles) issue_tile<MAPPED>(p, sm.tile[s], &sm.full[s], t, lane);
    }
  }

  const float sf = (float)p.s;
  const float cap = kTwo23 + sf;
  const uint32_t wpb = 1u << (p.log2d - 9);                      // warps per bucket
  const bool leader = (tid & (32u * wpb - 1u)) == 0;
  const uint32_t my_bucket = (tid * 16u) >> p.log2d;             // bucket of this thread in a tile
  const uint32_t buckets_per_tile_log2 = 12u - p.log2d;

  uint32_t stage = 0, phase = 0, it = 0;
  for (uint32_t t = blockIdx.x; t < p.full_tiles; t += grid, ++it) {
    const float* tile = sm.tile[stage];
    const bool arrived = mbar_wait_bounded(&sm.full[stage], phase, p.poll_limit);

    // ---- registers <- 16 consecutive coordinates; partial of the scale ----------------------
    float v[16];
#pragma unroll
    for (int j = 0; j < 4; ++j) {
      const float4 a = *reinterpret_cast<const float4*>(tile + tid * 16 + j * 4);
      v[4 * j] = a.x; v[4 * j + 1] = a.y; v[4 * j + 2] = a.z; v[4 * j + 3] = a.w;
    }
    float part = 0.f;
#pragma unroll
    for (int e = 0; e < 16; ++e) {
      if (NORM == QSGD_NORM_L2) part = fmaf(v[e], v[e], part);
      else part = fmaxf(part, fabsf(v[e]));
    }
    const float mine = part;                                       // this thread's share of the scale
#pragma unroll
    for (uint32_t o = 16; o > 0; o >>= 1) {
      const float q = __shfl_xor_sync(0xffffffffu, part, o);
      part = (NORM == QSGD_NORM_L2) ? part + q : fmaxf(part, q);
    }
    // 2-norm: an fp32 sum of squares outside [8e-28, 1e30] may have lost bits to underflow or
    // overflowed; such buckets are redone in fp64 (rare, the CTA branches together)
    bool shaky = false;
    // (a zero sum counts: squares below 1.4e-45 vanish in fp32 while the values do not in fp64)
    if (NORM == QSGD_NORM_L2) shaky = !(part >= 8.0e-28f && part <= 1.0e30f);
    if (lane == 0) sm.wsum[it & 1][warp] = part;

    // ---- release the stage: every warp signals that its values are in registers; the producer
    // thread refills the stage that was released one iteration ago (its arrivals are long in) ----
    __syncwarp();
    if (lane == 0) mbar_arrive(&sm.empty[stage]);
    // a wait that ran out ends the loop; the decision is taken per CTA (the scales meet in
    // shared memory), never per lane. __syncthreads_or tells only whether any thread's value was
    // nonzero, so the ordinary tile costs one barrier and an unusual one two more to tell a
    // timeout (bit 0) from a bucket that needs the fp64 path (bit 1).
    int flags = 0;
    if (__syncthreads_or((arrived ? 0 : 1) | (shaky ? 1 : 0)))
      flags = (__syncthreads_or(arrived ? 0 : 1) ? 1 : 0) | (__syncthreads_or(shaky ? 1 : 0) ? 2 : 0);
    if (flags & 1) {
      if (lane == 0) atomicOr(p.status, QSGD_DEV_TIMEOUT);
      break;
    }
    if (!MAPPED) {                                                        // ordinary case: thread 0 produces
      if (tid == 0 && it > 0) {
        const uint32_t ps = stage == 0 ? kStages - 1 : stage - 1;         // stage of iteration it - 1
        const uint32_t pphase = stage == 0 ? phase ^ 1 : phase;
        const uint32_t tn = t + (uint32_t)(kStages - 1) * grid;           // tile of iteration it - 1 + kStages
        if (tn < p.full_tiles) {
          if (mbar_wait_bounded(&sm.empty[ps], pphase, p.poll_limit)) issue_tile<false>(p, sm.tile[ps], &sm.full[ps], tn, 0u);
          else atomicOr(p.status, QSGD_DEV_TIMEOUT);
        }
      }
    } else if (warp == 0 && it > 0) {                                     // bucket map: warp 0 produces
      const uint32_t ps = stage == 0 ? kStages - 1 : stage - 1;
      const uint32_t pphase = stage == 0 ? phase ^ 1 : phase;
      const uint32_t tn = t + (uint32_t)(kStages - 1) * grid;
      if (tn < p.full_tiles) {
        const bool freed = __shfl_sync(0xffffffffu, lane == 0 ? (mbar_wait_bounded(&sm.empty[ps], pphase, p.poll_limit) ? 1 : 0) : 0, 0) != 0;
        __syncwarp();                                                     // lane 0's acquire covers the warp
        if (freed) issue_tile<true>(p, sm.tile[ps], &sm.full[ps], tn, lane);
        else if (lane == 0) atomicOr(p.status, QSGD_DEV_TIMEOUT);
      }
    }
    float A;
    bool clamp = true;
    {
      const uint32_t w0 = warp & ~(wpb - 1u);
      float acc = 0.f;
      for (uint32_t w = 0; w < wpb; ++w) {
        const float q = sm.wsum[it & 1][w0 + w];
        acc = (NORM == QSGD_NORM_L2) ? acc + q : fmaxf(acc, q);
      }
      if (NORM == QSGD_NORM_L2) {
        A = __fsqrt_rn(acc);
        // no per-coordinate clamp where no thread of the warp holds (nearly) all of its bucket's
        // sum of squares: see the per-warp kernel
        clamp = (flags & 2) || __any_sync(0xffffffffu, !(mine <= 0.9f * acc));
        if (flags & 2) {                      // some bucket of this tile needs the fp64 path
          double wide = 0.0;
#pragma unroll
          for (int e = 0; e < 16; ++e) wide = fma((double)v[e], (double)v[e], wide);
#pragma unroll
          for (int o = 16; o > 0; o >>= 1) wide += __shfl_xor_sync(0xffffffffu, wide, o);
          if (lane == 0) sm.wsum64[warp] = wide;
          __syncthreads();
          wide = 0.0;
          for (uint32_t w = 0; w < wpb; ++w) wide += sm.wsum64[w0 + w];
          A = __double2float_rn(sqrt(wide));
          __syncthreads();
        }
      } else {
        A = acc;
      }
    }
    if (!(A >= FLT_MIN)) A = 0.f;                      // zero bucket: Q(0) = 0
    const float r = A > 0.f ? __frcp_rn(A) : 0.f;
    if (leader) p.A_out[(t << buckets_per_tile_log2) + my_bucket] = A;

    // ---- stochastic rounding and packing ----------------------------------------------------
    float um[16];
    philox_uniforms16(t * (kTile / 4) + tid * 4, p.pc, um);
    uint32_t sw, lw[4];
    if (clamp) quantize16<LB, true>(v, um, r, sf, cap, lw, sw);
    else quantize16<LB, false>(v, um, r, sf, cap, lw, sw);
    if (LB != 8) sw &= nonzero_fields16<LB>(lw);          // canonical sign: 0 where the level is 0

    store_chunk<LB>(p.sign_out, p.level_out, t * (kTile / 512) + warp, lane, sw, lw);
    if (++stage == kStages) { stage = 0; phase ^= 1; }
  }

  // Leave no bulk copy in flight: a CTA that stopped early waits (bounded) for its ring.
  __syncthreads();
  if (tid == 0) {
    for (uint32_t j = 0; j < (uint32_t)kStages; ++j) {
      const uint32_t itj = it + j;
      const uint64_t t = (uint64_t)blockIdx.x + (uint64_t)itj * grid;
      if (t < p.full_tiles) mbar_wait_bounded(&sm.full[itj % kStages], (itj / kStages) & 1, kDrainPolls);
    }
  }
}

// ---------------------------------------------------------------------------------------------
// Generic kernel: any bucket size that is a multiple of 32. One CTA per tile of whole buckets.
// ---------------------------------------------------------------------------------------------
constexpr int kGroupsPerThread = kTile / 8 / kThreads;  // 2
constexpr int kMaxBucketsPerTile = kTile / 32;          // 128

// One tile of the generic path. `block` / `nblocks` play the role of blockIdx / gridDim so that the
// main kernel can run the ragged last tile in one extra CTA of its own grid.
template <int LB, int NORM, bool MAPPED>
__device__ __forceinline__ void quantize_generic_tile(const QuantizeParams& p, uint32_t block, uint32_t nblocks,
                                                      float* tile, float* part, float* s_rcp) {
  const uint32_t tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const uint64_t t0 = p.coord_base + (uint64_t)block * p.tile_coords;   // first coordinate
  if (block == 0 && tid == 0 && p.info) {
    p.info[0] = 8 * p.total_bytes; p.info[1] = 0; p.info[2] = p.total_bytes; p.info[3] = 0;
  }
  if (block == 0 && tid == 0 && p.clear_word) *p.clear_word = 0u;
  const uint64_t left = p.n - t0;
  const uint32_t valid = left < p.tile_coords ? (uint32_t)left : p.tile_coords;
  if (valid == 0) {                            // nothing left to encode: only the padding
    if (tid < 4) {
      if (p.B + tid < ((p.B + 3) & ~3ull)) p.A_out[p.B + tid] = 0.f;
      if (p.sign_words + tid < ((p.sign_words + 3) & ~3ull)) p.sign_out[p.sign_words + tid] = 0u;
      if (p.level_words + tid < ((p.level_words + 3) & ~3ull)) p.level_out[p.level_words + tid] = 0u;
    }
    return;
  }

  for (uint32_t i = tid * 4; i < p.tile_coords; i += kThreads * 4) {
    float4 v = make_float4(0.f, 0.f, 0.f, 0.f);
    if (MAPPED) {
      // per-tensor policy: four coordinates of one bucket (d is a multiple of 32) from the
      // bucket's own place; what lies behind the bucket's length is zero padding
      if (i < valid) {
        const uint32_t bi = i / p.d, c = i - bi * p.d;
        const uint64_t b = t0 / p.d + bi;
        const uint32_t L = __ldg(p.map.len + b);
        const float* src = p.g + __ldg(p.map.src + b) + c;
        if (c + 4 <= L && (reinterpret_cast<uintptr_t>(src) & 15u) == 0) {
          v = __ldcs(reinterpret_cast<const float4*>(src));
        } else {
          float t[4] = {0.f, 0.f, 0.f, 0.f};
          for (uint32_t j = 0; j < 4 && c + j < L; ++j) t[j] = src[j];
          v = make_float4(t[0], t[1], t[2], t[3]);
        }
      }
    } else if (i + 4 <= valid) {
      v = __ldcs(reinterpret_cast<const float4*>(p.g + t0 + i));
    } else if (i < valid) {
      float t[4] = {0.f, 0.f, 0.f, 0.f};
      for (uint32_t j = 0; i + j < valid; ++j) t[j] = p.g[t0 + i + j];
      v = make_float4(t[0], t[1], t[2], t[3]);
    }
    *reinterpret_cast<float4*>(tile + i) = v;
  }
  __syncthreads();

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

  const uint32_t nb = p.tile_coords / p.d;     // buckets in a full tile
  const uint32_t gpb = p.d >> 3;               // groups per bucket
  const uint64_t b0 = t0 / p.d;                // first bucket of the tile
  for (uint32_t b = warp; b < nb; b += kThreads / 32) {
    float A;
    if (NORM == QSGD_NORM_L2) {
      // fp32 partials of 8 squares each; redo in fp64 from the tile when they may have lost bits:
      // a nonzero partial outside [8e-28, 1e30], or a bucket total below that range (a zero total
      // too: squares below 1.4e-45 vanish in fp32 while the values do not in fp64)
      double acc = 0.0;
      bool shaky = false;
      for (uint32_t j = lane; j < gpb; j += 32) {
        const float q = part[b * gpb + j];
        shaky |= !(q >= 8.0e-28f && q <= 1.0e30f) && q != 0.f;
        acc += (double)q;
      }
#pragma unroll
      for (int o = 16; o > 0; o >>= 1) acc += __shfl_xor_sync(0xffffffffu, acc, o);
      if (__any_sync(0xffffffffu, shaky) || !(acc >= 8.0e-28)) {
        acc = 0.0;
        for (uint32_t i = lane; i < p.d; i += 32) {
          const double x = (double)tile[b * p.d + i];
          acc = fma(x, x, acc);
        }
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) acc += __shfl_xor_sync(0xffffffffu, acc, o);
      }
      A = __double2float_rn(__dsqrt_rn(acc));
    } else {
      float acc = 0.f;
      for (uint32_t j = lane; j < gpb; j += 32) acc = fmaxf(acc, part[b * gpb + j]);
#pragma unroll
      for (int o = 16; o > 0; o >>= 1) acc = fmaxf(acc, __shfl_xor_sync(0xffffffffu, acc, o));
      A = acc;
    }
    if (!(A >= FLT_MIN)) A = 0.f;
    if (lane == 0) {
      s_rcp[b] = A > 0.f ? __frcp_rn(A) : 0.f;
      if (b0 + b < p.B) p.A_out[b0 + b] = A;
    }
  }
  __syncthreads();

  const float sf = (float)p.s;
#pragma unroll
  for (int j = 0; j < kGroupsPerThread; ++j) {
    const uint32_t grp = tid + j * kThreads;
    const uint32_t bl = (grp * 8) / p.d;
    const float r = (grp < groups) ? s_rcp[bl] : 0.f;
    const uint64_t i0 = t0 + (uint64_t)grp * 8;
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

  if (block == nblocks - 1 && tid < 4) {
    if (p.B + tid < ((p.B + 3) & ~3ull)) p.A_out[p.B + tid] = 0.f;
    if (p.sign_words + tid < ((p.sign_words + 3) & ~3ull)) p.sign_out[p.sign_words + tid] = 0u;
    if (p.level_words + tid < ((p.level_words + 3) & ~3ull)) p.level_out[p.level_words + tid] = 0u;
  }
}

// ---------------------------------------------------------------------------------------------
// Per-warp streaming kernel: d <= 512 (a bucket never leaves a warp).
// Warp w of CTA b takes chunks b * 8 + w, + 8 * main_ctas, ... of 512 coordinates. Its ring of
// kWarpStages stages is private: lane 0 arms a stage (expect-tx + bulk copy), all lanes wait on
// the stage's barrier, pull their 16 values into registers, and after the shuffle reduction of
// the scale (which cannot finish before every lane's values have arrived) lane 0 re-arms the
// stage for the chunk kWarpStages rounds ahead. One optional extra CTA runs the ragged last
// tile and the region padding through the generic tile code.
// ---------------------------------------------------------------------------------------------
constexpr int kWarpStages = 3;
constexpr int kChunk = 512;

struct __align__(16) WarpRings {
  float chunk[kThreads / 32][kWarpStages][kChunk];
  uint64_t full[kThreads / 32][kWarpStages];
};

// How the per-warp kernel finds its chunks. The streaming loop is sensitive to every warp-wide step
// added to it (a shuffle and a vote on the map entries cost 8 % of the kernel's time with nothing
// else changed), so with a map every lane that owns a bucket of the chunk starts that bucket's copy
// by itself, and the zeros behind a short bucket are one more copy, from a block of zeros in global
// memory: no loop, no call, no common step. Buckets of 512 -- one per chunk, lane 0 alone at work --
// are an instantiation of their own. What is left of the map's cost is about 8 % against the same
// buckets without a map (6 % of it gone when the entries are computed instead of loaded).
enum MapMode { kNoMap = 0, kMapOnePerChunk = 1, kMapSeveralPerChunk = 2 };

__device__ __align__(128) float g_zero_chunk[kChunk];      // never written

// What lane j < 512 / d knows of bucket j of a chunk when buckets come through a bucket map.
struct MappedBucket {
  uint64_t src;   // first coordinate of the bucket in g
  uint32_t len;   // coordinates it holds (<= d; zeros stand behind a short one)
};

template <int MAP>
__device__ __forceinline__ MappedBucket fetch_bucket(const FastParams& p, uint32_t chunk, uint32_t chunks,
                                                     uint32_t lane) {
  MappedBucket mb{0ull, 0u};
  if (MAP != kNoMap) {
    const uint32_t nb = (uint32_t)kChunk >> p.log2d;
    if (chunk < chunks && lane < nb) {
      const uint64_t b = ((uint64_t)chunk << (9u - p.log2d)) + lane;
      mb.src = __ldg(p.map.src + b);
      mb.len = min(__ldg(p.map.len + b), 1u << p.log2d);
    }
  }
  return mb;
}

// Arm one stage for `chunk` (called by the whole warp; its reads of the stage are already done).
// The stage always receives kChunk * 4 bytes: lane 0 announces them, and the copies may complete
// before or after that (the barrier's transaction count is signed). The map guarantees 16-byte
// aligned places and lengths.
template <int MAP>
__device__ __forceinline__ void arm_chunk(const FastParams& p, float* dst, uint64_t* bar, uint32_t chunk,
                                          uint32_t lane, const MappedBucket mb) {
  if (MAP == kNoMap) {
    if (lane == 0) {
      asm volatile("fence.proxy.async.shared::cta;" ::: "memory");     // our reads before the copy's writes
      mbar_expect_tx(bar, kChunk * 4);
      bulk_load(dst, p.g + (size_t)chunk * kChunk, kChunk * 4, bar);
    }
    return;
  }
  const uint32_t d = MAP == kMapOnePerChunk ? (uint32_t)kChunk : 1u << p.log2d;
  const uint32_t nb = MAP == kMapOnePerChunk ? 1u : (uint32_t)kChunk >> p.log2d;
  if (lane < nb) {
    asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
    if (lane == 0) mbar_expect_tx(bar, kChunk * 4);
    float* mine = dst + lane * d;
    if (mb.len) bulk_load(mine, p.g + mb.src, 4u * mb.len, bar);
    if (mb.len != d) bulk_load(mine + mb.len, g_zero_chunk, 4u * (d - mb.len), bar);
  }
}

template <int LB, int NORM, int MAP>
__global__ void __launch_bounds__(kThreads, 4)
quantize_warp_kernel(const __grid_constant__ FastParams p) {
  extern __shared__ __align__(128) uint8_t smem_raw[];
  WarpRings& sm = *reinterpret_cast<WarpRings*>(smem_raw);
  const uint32_t tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const uint32_t grid = p.main_ctas;
  if (blockIdx.x >= grid) {                     // the extra CTA: ragged tail + padding
    chain_wait();
    float* scratch = &sm.chunk[0][0][0];
    quantize_generic_tile<LB, NORM, MAP != kNoMap>(p.tail, 0u, 1u, scratch, scratch + kTile, scratch + kTile + 1024);
    return;
  }
  const uint32_t chunks = p.full_tiles * (kTile / kChunk), stride = grid * (kThreads / 32);
  uint32_t c = blockIdx.x * (kThreads / 32) + warp;
  if (lane == 0) {
    for (int s = 0; s < kWarpStages; ++s) mbar_init(&sm.full[warp][s], 1);
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  chain_wait();                                 // nothing above touches global memory
  if (tid == 0 && blockIdx.x == 0) {
    if (p.info) { p.info[0] = 8 * p.total_bytes; p.info[1] = 0; p.info[2] = p.total_bytes; p.info[3] = 0; }
    if (p.clear_word) *p.clear_word = 0u;
  }
  __syncwarp();
  for (int s = 0; s < kWarpStages; ++s) {
    const uint32_t cs = c + (uint32_t)s * stride;
    if (cs < chunks) {
      const MappedBucket mb = fetch_bucket<MAP>(p, cs, chunks, lane);
      arm_chunk<MAP>(p, sm.chunk[warp][s], &sm.full[warp][s], cs, lane, mb);
    }
  }
  // the map entries of the next chunk to arm are fetched one round ahead of their use
  MappedBucket ahead = fetch_bucket<MAP>(p, c + (uint32_t)kWarpStages * stride, chunks, lane);

  const float sf = (float)p.s;
  const float cap = kTwo23 + sf;
  const uint32_t team_w = 1u << (p.log2d - 4);                   // lanes per bucket (2 .. 32)
  const bool leader = (lane & (team_w - 1u)) == 0;
  const uint32_t my_bucket = (lane * 16u) >> p.log2d;            // bucket of this lane in a chunk
  const uint32_t buckets_per_chunk_log2 = 9u - p.log2d;

  uint32_t stage = 0, phase = 0;
  for (; c < chunks; c += stride) {
    const float* src = sm.chunk[warp][stage];
    const bool arrived = mbar_wait_bounded(&sm.full[warp][stage], phase, p.poll_limit);
    if (!__all_sync(0xffffffffu, arrived)) {                       // the warp leaves together
      if (lane == 0) atomicOr(p.status, QSGD_DEV_TIMEOUT);
      break;
    }

    // ---- registers <- 16 consecutive coordinates; the uniforms; partial of the scale ---------
    float v[16];
#pragma unroll
    for (int j = 0; j < 4; ++j) {
      const float4 a = *reinterpret_cast<const float4*>(src + lane * 16 + j * 4);
      v[4 * j] = a.x; v[4 * j + 1] = a.y; v[4 * j + 2] = a.z; v[4 * j + 3] = a.w;
    }
    // Where the uniforms are computed does not change the work, only what the compiler makes of the
    // loop, and that was measured: ahead of the scale reduction with the 2-norm (75 against 80 us at
    // s = 255), behind it with the max-norm (78 against 86 us at s = 255, 79 against 82 at s = 15).
    constexpr bool kUniformsLate = NORM == QSGD_NORM_MAX;
    float um[16];
    if (!kUniformsLate) philox_uniforms16(c * (kChunk / 4) + lane * 4, p.pc, um);
    float part = 0.f;
#pragma unroll
    for (int e = 0; e < 16; ++e) {
      if (NORM == QSGD_NORM_L2) part = fmaf(v[e], v[e], part);
      else part = fmaxf(part, fabsf(v[e]));
    }
    const float mine = part;                                       // this thread's share of the scale
    if (team_w == 32u) {
#pragma unroll
      for (uint32_t o = 16; o > 0; o >>= 1) {
        const float q = __shfl_xor_sync(0xffffffffu, part, o);
        part = (NORM == QSGD_NORM_L2) ? part + q : fmaxf(part, q);
      }
    } else {
#pragma unroll
      for (uint32_t o = 16; o > 0; o >>= 1) {
        const float q = __shfl_xor_sync(0xffffffffu, part, o);
        const float merged = (NORM == QSGD_NORM_L2) ? part + q : fmaxf(part, q);
        part = (o < team_w) ? merged : part;
      }
    }

    // ---- the stage is in registers: refill it with the chunk kWarpStages rounds ahead --------
    __syncwarp();
    {
      const uint32_t cn = c + (uint32_t)kWarpStages * stride;
      if (cn < chunks) arm_chunk<MAP>(p, sm.chunk[warp][stage], &sm.full[warp][stage], cn, lane, ahead);
      ahead = fetch_bucket<MAP>(p, cn + stride, chunks, lane);
    }

    // ---- scale ---------------------------------------------------------------------------------
    // 2-norm: an fp32 sum of squares outside [8e-28, 1e30] may have lost bits to underflow or
    // overflowed; such buckets are redone in fp64 (rare, the warp branches together)
    float A;
    bool shaky = false;
    if (NORM == QSGD_NORM_L2) {
      shaky = !(part >= 8.0e-28f && part <= 1.0e30f);   // a zero sum too: tiny squares vanish in fp32
      A = __fsqrt_rn(part);
      if (__any_sync(0xffffffffu, shaky)) {
        double wide = 0.0;
#pragma unroll
        for (int e = 0; e < 16; ++e) wide = fma((double)v[e], (double)v[e], wide);
#pragma unroll
        for (uint32_t o = 16; o > 0; o >>= 1) {
          const double q = __shfl_xor_sync(0xffffffffu, wide, o);
          wide = (o < team_w) ? wide + q : wide;
        }
        if (shaky) A = __double2float_rn(sqrt(wide));
      }
    } else {
      A = part;
    }
    if (!(A >= FLT_MIN)) A = 0.f;                      // zero bucket: Q(0) = 0
    const float r = A > 0.f ? __frcp_rn(A) : 0.f;
    if (leader) p.A_out[(c << buckets_per_chunk_log2) + my_bucket] = A;

    // ---- stochastic rounding and packing -------------------------------------------------------
    // floor(t + u) can pass s only where t = (s |v|) / A reaches s, i.e. |v| is A up to rounding.
    // With the 2-norm that needs one coordinate to hold (nearly) all of the bucket's sum of
    // squares; a thread whose 16 squares stay under 0.9 of the sum holds no such coordinate, and
    // a warp of such threads rounds without the clamp. (Not so for the max-norm, where the
    // largest coordinate always has |v| = A.)
    if (kUniformsLate) philox_uniforms16(c * (kChunk / 4) + lane * 4, p.pc, um);
    uint32_t sw, lw[4];
    bool clamp = true;
    if (NORM == QSGD_NORM_L2) clamp = __any_sync(0xffffffffu, shaky || !(mine <= 0.9f * part));
    if (clamp) quantize16<LB, true>(v, um, r, sf, cap, lw, sw);
    else quantize16<LB, false>(v, um, r, sf, cap, lw, sw);
    if (LB != 8) sw &= nonzero_fields16<LB>(lw);          // canonical sign: 0 where the level is 0
    store_chunk<LB>(p.sign_out, p.level_out, c, lane, sw, lw);
    if (++stage == kWarpStages) { stage = 0; phase ^= 1; }
  }

  // Leave no bulk copy in flight: a warp that stopped early waits (bounded) for the stages it armed.
  if (lane == 0 && c < chunks) {
    for (uint32_t j = 0; j < (uint32_t)kWarpStages; ++j) {
      if (c + j * stride < chunks) mbar_wait_bounded(&sm.full[warp][stage], phase, kDrainPolls);
      if (++stage == kWarpStages) { stage = 0; phase ^= 1; }
    }
  }
}

// ---------------------------------------------------------------------------------------------
// Per-warp pipelines for d >= 1024: a bucket is 2^(log2d - 9) consecutive chunks, taken by as
// many neighbouring warps of one CTA (a group). Each warp streams its chunk exactly as in
// quantize_warp_kernel; once per chunk the group's warps meet at a named barrier of their own to
// exchange their partial sums (and the "my wait ran out" / "my sum left the fp32 range" flags, so
// that the whole group takes the same path). No CTA-wide barrier, no producer thread.
// ---------------------------------------------------------------------------------------------
struct __align__(16) GroupRings {
  WarpRings rings;
  float wsum[2][kThreads / 32];
  uint32_t wflag[2][kThreads / 32];
  double wsum64[kThreads / 32];
};

__device__ __forceinline__ void group_barrier(uint32_t id, uint32_t threads) {
  asm volatile("bar.sync %0, %1;" ::"r"(id), "r"(threads) : "memory");
}

// With a bucket map: the piece of bucket (chunk / chunks-per-bucket) that this chunk covers.
template <bool MAPPED>
__device__ __forceinline__ MappedBucket fetch_piece(const FastParams& p, uint32_t chunk, uint32_t chunks,
                                                    uint32_t lane) {
  MappedBucket mb{0ull, 0u};
  if (MAPPED && chunk < chunks && lane == 0) {
    const uint32_t sh = p.log2d - 9u;
    const uint64_t b = chunk >> sh;
    const uint32_t off = (chunk & ((1u << sh) - 1u)) << 9;
    const uint32_t L = min(__ldg(p.map.len + b), 1u << p.log2d);
    mb.src = __ldg(p.map.src + b) + off;
    mb.len = L > off ? min(L - off, (uint32_t)kChunk) : 0u;
  }
  return mb;
}

template <int LB, int NORM, bool MAPPED>
__global__ void __launch_bounds__(kThreads, 4)
quantize_group_kernel(const __grid_constant__ FastParams p) {
  extern __shared__ __align__(128) uint8_t smem_raw[];
  GroupRings& gs = *reinterpret_cast<GroupRings*>(smem_raw);
  WarpRings& sm = gs.rings;
  constexpr int MAP = MAPPED ? kMapOnePerChunk : kNoMap;
  const uint32_t tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const uint32_t grid = p.main_ctas;
  if (blockIdx.x >= grid) {                     // the extra CTA: ragged tail + padding
    chain_wait();
    float* scratch = &sm.chunk[0][0][0];
    quantize_generic_tile<LB, NORM, MAPPED>(p.tail, 0u, 1u, scratch, scratch + kTile, scratch + kTile + 1024);
    return;
  }
  const uint32_t chunks = p.full_tiles * (kTile / kChunk), stride = grid * (kThreads / 32);
  uint32_t c = blockIdx.x * (kThreads / 32) + warp;
  if (lane == 0) {
    for (int s = 0; s < kWarpStages; ++s) mbar_init(&sm.full[warp][s], 1);
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  chain_wait();                                 // nothing above touches global memory
  if (tid == 0 && blockIdx.x == 0) {
    if (p.info) { p.info[0] = 8 * p.total_bytes; p.info[1] = 0; p.info[2] = p.total_bytes; p.info[3] = 0; }
    if (p.clear_word) *p.clear_word = 0u;
  }
  __syncwarp();
  for (int s = 0; s < kWarpStages; ++s) {
    const uint32_t cs = c + (uint32_t)s * stride;
    if (cs < chunks) {
      const MappedBucket mb = fetch_piece<MAPPED>(p, cs, chunks, lane);
      arm_chunk<MAP>(p, sm.chunk[warp][s], &sm.full[warp][s], cs, lane, mb);
    }
  }
  MappedBucket ahead = fetch_piece<MAPPED>(p, c + (uint32_t)kWarpStages * stride, chunks, lane);

  const float sf = (float)p.s;
  const float cap = kTwo23 + sf;
  const uint32_t wpb = 1u << (p.log2d - 9);                      // warps per bucket = warps of a group
  const uint32_t w0 = warp & ~(wpb - 1u);                        // first warp of this warp's group
  const uint32_t bar_id = 1u + (w0 >> (p.log2d - 9));            // named barriers 1 .. 4
  const bool leader = warp == w0 && lane == 0;

  uint32_t stage = 0, phase = 0, it = 0;
  for (; c < chunks; c += stride, ++it) {
    const float* src = sm.chunk[warp][stage];
    const bool ok = __all_sync(0xffffffffu, mbar_wait_bounded(&sm.full[warp][stage], phase, p.poll_limit));

    float v[16];
#pragma unroll
    for (int j = 0; j < 4; ++j) {
      const float4 a = *reinterpret_cast<const float4*>(src + lane * 16 + j * 4);
      v[4 * j] = a.x; v[4 * j + 1] = a.y; v[4 * j + 2] = a.z; v[4 * j + 3] = a.w;
    }
    float um[16];
    philox_uniforms16(c * (kChunk / 4) + lane * 4, p.pc, um);
    float part = 0.f;
#pragma unroll
    for (int e = 0; e < 16; ++e) {
      if (NORM == QSGD_NORM_L2) part = fmaf(v[e], v[e], part);
      else part = fmaxf(part, fabsf(v[e]));
    }
    const float mine = part;
#pragma unroll
    for (uint32_t o = 16; o > 0; o >>= 1) {
      const float q = __shfl_xor_sync(0xffffffffu, part, o);
      part = (NORM == QSGD_NORM_L2) ? part + q : fmaxf(part, q);
    }
    bool shaky = false;
    if (NORM == QSGD_NORM_L2) shaky = !(part >= 8.0e-28f && part <= 1.0e30f);   // a zero sum too
    const uint32_t par = it & 1u;
    if (lane == 0) {
      gs.wsum[par][warp] = part;
      gs.wflag[par][warp] = (ok ? 0u : 1u) | (shaky ? 2u : 0u);
    }

    // ---- the stage is in registers: refill it (not after a wait that ran out: its copy may still land)
    __syncwarp();
    {
      const uint32_t cn = c + (uint32_t)kWarpStages * stride;
      if (ok && cn < chunks) arm_chunk<MAP>(p, sm.chunk[warp][stage], &sm.full[warp][stage], cn, lane, ahead);
      ahead = fetch_piece<MAPPED>(p, cn + stride, chunks, lane);
    }

    // ---- the group's warps exchange their sums ---------------------------------------------------
    group_barrier(bar_id, 32u * wpb);
    float acc = 0.f;
    uint32_t fl = 0u;
    for (uint32_t w = 0; w < wpb; ++w) {
      const float q = gs.wsum[par][w0 + w];
      acc = (NORM == QSGD_NORM_L2) ? acc + q : fmaxf(acc, q);
      fl |= gs.wflag[par][w0 + w];
    }
    float A;
    if (NORM == QSGD_NORM_L2) {
      A = __fsqrt_rn(acc);
      if (fl & 2u) {                          // some warp's sum left the fp32 range: the bucket again in fp64
        double wide = 0.0;
#pragma unroll
        for (int e = 0; e < 16; ++e) wide = fma((double)v[e], (double)v[e], wide);
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) wide += __shfl_xor_sync(0xffffffffu, wide, o);
        if (lane == 0) gs.wsum64[warp] = wide;
        group_barrier(bar_id, 32u * wpb);
        wide = 0.0;
        for (uint32_t w = 0; w < wpb; ++w) wide += gs.wsum64[w0 + w];
        A = __double2float_rn(sqrt(wide));
        group_barrier(bar_id, 32u * wpb);
      }
    } else {
      A = acc;
    }
    if (!ok) {                                 // this warp's wait ran out: it leaves with its stage still armed
      if (lane == 0) atomicOr(p.status, QSGD_DEV_TIMEOUT);
      break;
    }
    if (!(A >= FLT_MIN)) A = 0.f;                      // zero bucket: Q(0) = 0
    const float r = A > 0.f ? __frcp_rn(A) : 0.f;
    if (leader) p.A_out[c >> (p.log2d - 9)] = A;

    uint32_t sw, lw[4];
    bool clamp = true;
    if (NORM == QSGD_NORM_L2) clamp = (fl & 2u) || __any_sync(0xffffffffu, !(mine <= 0.9f * acc));
    if (clamp) quantize16<LB, true>(v, um, r, sf, cap, lw, sw);
    else quantize16<LB, false>(v, um, r, sf, cap, lw, sw);
    if (LB != 8) sw &= nonzero_fields16<LB>(lw);          // canonical sign: 0 where the level is 0
    store_chunk<LB>(p.sign_out, p.level_out, c, lane, sw, lw);
    if (++stage == kWarpStages) { stage = 0; phase ^= 1; }
    if (fl & 1u) { c += stride; break; }       // another warp of the group gave up: the group stops together
  }

  // Leave no bulk copy in flight: a warp that stopped early waits (bounded) for the stages it armed.
  if (lane == 0 && c < chunks) {
    for (uint32_t j = 0; j < (uint32_t)kWarpStages; ++j) {
      if (c + j * stride < chunks) mbar_wait_bounded(&sm.full[warp][stage], phase, kDrainPolls);
      if (++stage == kWarpStages) { stage = 0; phase ^= 1; }
    }
  }
}

template <int LB, int NORM, bool MAPPED>
__global__ void __launch_bounds__(kThreads) quantize_generic_kernel(const QuantizeParams p) {
  __shared__ __align__(16) float tile[kTile];
  __shared__ float part[kTile / 8];
  __shared__ float s_rcp[kMaxBucketsPerTile];
  chain_wait();
  quantize_generic_tile<LB, NORM, MAPPED>(p, blockIdx.x, gridDim.x, tile, part, s_rcp);
}

PhiloxConsts make_philox_consts(uint64_t seed, uint32_t step, uint32_t worker) {
  uint32_t k0[10], k1[10];
  k0[0] = (uint32_t)seed; k1[0] = (uint32_t)(seed >> 32);
  for (int r = 1; r < 10; ++r) { k0[r] = k0[r - 1] + 0x9E3779B9u; k1[r] = k1[r - 1] + 0xBB67AE85u; }
  const uint64_t ps = (uint64_t)kM1 * step;
  const uint32_t x0 = (uint32_t)(ps >> 32) ^ k0[0], l1 = (uint32_t)ps;
  const uint64_t px = (uint64_t)kM0 * x0;
  PhiloxConsts pc;
  pc.y0 = worker ^ k1[0];
  pc.z0 = l1 ^ k0[1];
  pc.z1 = (uint32_t)(px >> 32) ^ k1[1];
  pc.z2 = (uint32_t)px ^ k1[2];
  pc.k0_2 = k0[2];
  for (int r = 0; r < 7; ++r) { pc.k[r][0] = k0[r + 3]; pc.k[r][1] = k1[r + 3]; }
  return pc;
}

std::atomic<uint32_t> g_poll_limit{kDrainPolls};

template <int LB, int NORM, int MAP>
int launch_warp(FastParams& fp, bool with_tail, cudaStream_t stream) {
  static KernelSite site;
  const size_t smem = sizeof(WarpRings) + 128;
  int sms = 0, ctas_per_sm = 0;
  const int st = site.lookup(quantize_warp_kernel<LB, NORM, MAP>, kThreads, smem, &sms, &ctas_per_sm);
  if (st) return st;
  const uint32_t cap = (uint32_t)(sms * ctas_per_sm);
  fp.main_ctas = fp.full_tiles < cap ? fp.full_tiles : cap;
  fp.poll_limit = g_poll_limit.load(std::memory_order_relaxed);
  ScopedKernel sk(kKernQuantize, stream);
  return (int)launch_chained(quantize_warp_kernel<LB, NORM, MAP>, fp.main_ctas + (with_tail ? 1u : 0u), kThreads, smem,
                             stream, fp);
}

template <int LB, int NORM, bool MAPPED>
int launch_group(FastParams& fp, bool with_tail, cudaStream_t stream) {
  static KernelSite site;
  const size_t smem = sizeof(GroupRings) + 128;
  int sms = 0, ctas_per_sm = 0;
  const int st = site.lookup(quantize_group_kernel<LB, NORM, MAPPED>, kThreads, smem, &sms, &ctas_per_sm);
  if (st) return st;
  const uint32_t cap = (uint32_t)(sms * ctas_per_sm);
  fp.main_ctas = fp.full_tiles < cap ? fp.full_tiles : cap;
  fp.poll_limit = g_poll_limit.load(std::memory_order_relaxed);
  ScopedKernel sk(kKernQuantize, stream);
  return (int)launch_chained(quantize_group_kernel<LB, NORM, MAPPED>, fp.main_ctas + (with_tail ? 1u : 0u), kThreads, smem,
                             stream, fp);
}

// d >= 1024, max-norm or bucket map: the CTA-wide ring.
template <int LB, int NORM, bool MAPPED>
int launch_cross(FastParams& fp, bool with_tail, cudaStream_t stream) {
  static KernelSite site;
  const size_t smem = sizeof(TileSmem) + 128;
  int sms = 0, ctas_per_sm = 0;
  const int st = site.lookup(quantize_pow2_kernel<LB, NORM, MAPPED>, kThreads, smem, &sms, &ctas_per_sm);
  if (st) return st;
  const uint32_t cap = (uint32_t)(sms * ctas_per_sm);
  fp.main_ctas = fp.full_tiles < cap ? fp.full_tiles : cap;
  fp.poll_limit = g_poll_limit.load(std::memory_order_relaxed);
  ScopedKernel sk(kKernQuantize, stream);
  return (int)launch_chained(quantize_pow2_kernel<LB, NORM, MAPPED>, fp.main_ctas + (with_tail ? 1u : 0u), kThreads, smem,
                             stream, fp);
}

template <int LB, int NORM>
int launch_one(QuantizeParams& p, uint64_t seed, cudaStream_t stream) {
  const uint32_t d = p.d;
  const bool pow2 = (d & (d - 1)) == 0;
  uint32_t full_tiles = 0;
  // with a bucket map the bulk copies need 16-byte aligned places and lengths
  const bool map_ok = !p.map.src || p.map.quads != 0u;
  if (pow2 && p.n <= (1ull << 32) && map_ok) full_tiles = (uint32_t)(p.n / kTile);
  if (full_tiles > 0) {
    FastParams fp;
    fp.g = p.g; fp.full_tiles = full_tiles; fp.s = p.s;
    fp.log2d = 0;
    while ((1u << fp.log2d) < d) ++fp.log2d;
    fp.A_out = p.A_out; fp.sign_out = p.sign_out; fp.level_out = p.level_out; fp.status = p.status;
    fp.info = p.info; fp.total_bytes = p.total_bytes; fp.clear_word = p.clear_word;
    fp.pc = make_philox_consts(seed, p.step, p.worker);
    fp.map = p.map;
    // the ragged tail (fewer than 4096 coordinates) and the zero padding of the three regions go
    // to one extra CTA of the same launch; nothing to do when n is a multiple of the tile and
    // every region already ends on a 16-byte boundary
    p.coord_base = (uint64_t)full_tiles * kTile;
    const bool with_tail = !(p.n == p.coord_base && ((p.B | p.sign_words | p.level_words) & 3ull) == 0);
    fp.tail = p;
    fp.tail.info = nullptr;
    fp.tail.clear_word = nullptr;
    if (d >= 1024) {
      // measured (n = 60 M, s = 15 / 255): with the 2-norm the per-warp pipelines with group barriers
      // take 83-86 us against the CTA-wide ring's 90-92; with the max-norm (100 against 84) and under a
      // bucket map (101 against 97) the ring is the faster one
      if constexpr (NORM == QSGD_NORM_L2) {
        if (!fp.map.src) return launch_group<LB, NORM, false>(fp, with_tail, stream);
      }
      return fp.map.src ? launch_cross<LB, NORM, true>(fp, with_tail, stream)
                        : launch_cross<LB, NORM, false>(fp, with_tail, stream);
    }
    if (!fp.map.src) return launch_warp<LB, NORM, kNoMap>(fp, with_tail, stream);
    return d == (uint32_t)kChunk ? launch_warp<LB, NORM, kMapOnePerChunk>(fp, with_tail, stream)
                                 : launch_warp<LB, NORM, kMapSeveralPerChunk>(fp, with_tail, stream);
  }
  // the fast path does not apply: everything through the generic kernel
  p.coord_base = 0;
  const uint64_t rem = p.n;
  uint64_t tiles = (rem + p.tile_coords - 1) / p.tile_coords;
  if (tiles == 0) tiles = 1;
  {
    ScopedKernel sk(kKernQuantizeTail, stream);
    if (p.map.src) return (int)launch_chained(quantize_generic_kernel<LB, NORM, true>, (uint32_t)tiles, kThreads, 0, stream, p);
    return (int)launch_chained(quantize_generic_kernel<LB, NORM, false>, (uint32_t)tiles, kThreads, 0, stream, p);
  }
}

template <int LB>
int launch_lb(QuantizeParams& p, int norm_kind, uint64_t seed, cudaStream_t stream) {
  return norm_kind == QSGD_NORM_L2 ? launch_one<LB, QSGD_NORM_L2>(p, seed, stream)
                                   : launch_one<LB, QSGD_NORM_MAX>(p, seed, stream);
}

}  // namespace

int launch_quantize_fixed(const float* g, uint64_t n, uint32_t d, uint32_t s, int norm_kind,
                          uint64_t seed, uint32_t step, uint32_t worker, uint8_t* out,
                          uint32_t* status_dev, uint64_t* info, uint32_t* clear_word, const BucketMap& map,
                          cudaStream_t stream) {
  const FixedLayout L = make_fixed_layout(n, d, s);
  QuantizeParams p;
  p.g = g; p.n = n; p.d = d; p.s = s; p.map = map;
  p.tile_coords = (kTile / d) * d;
  p.coord_base = 0;
  p.k0 = (uint32_t)seed; p.k1 = (uint32_t)(seed >> 32); p.step = step; p.worker = worker;
  p.A_out = reinterpret_cast<float*>(out);
  p.sign_out = reinterpret_cast<uint32_t*>(out + L.off_sign);
  p.level_out = reinterpret_cast<uint32_t*>(out + L.off_level);
  p.B = L.B; p.sign_words = L.sign_words; p.level_words = L.level_words;
  p.tiles = 0;
  p.status = status_dev;
  p.info = info;
  p.total_bytes = L.total;
  p.clear_word = clear_word;
  switch (L.lb) {
    case 1: return launch_lb<1>(p, norm_kind, seed, stream);
    case 2: return launch_lb<2>(p, norm_kind, seed, stream);
    case 4: return launch_lb<4>(p, norm_kind, seed, stream);
    default: return launch_lb<8>(p, norm_kind, seed, stream);
  }
}

void set_quantize_poll_limit(uint32_t polls) { g_poll_limit.store(polls, std::memory_order_relaxed); }
uint32_t default_quantize_poll_limit() { return kDrainPolls; }

}  // namespace qsgd
