// Encode, Elias path (Section 3.1 "Efficient Coding of Gradients", string S; Appendix A.3 for
// the dense variant). Pipeline on one stream:
//   1. quantize into the fixed-width layout held in the workspace (quantize_fixed.cu);
//   2. string length L_b of every bucket, and the sum of the lengths of each CTA's run of
//      consecutive buckets (elias_length_kernel);
//   3. the CTA of the length kernel that publishes its sum last (an arrival counter, no waiting)
//      scans the per-CTA sums, fixes the message geometry, checks the capacity and clears the few
//      payload words that two scatter CTAs will share;
//   4. each CTA of the scatter kernel derives the bit offsets of its own buckets, writes their
//      offset-table entries, assembles its run of strings in shared memory (lanes own
//      consecutive sub-ranges of a bucket; bits of neighbouring lanes and buckets meet inside
//      words and are merged with shared-memory atomics) and flushes whole words to the payload
//      with coalesced stores; only the first and last word of a CTA's range, which it may share
//      with its neighbours, are merged with atomicOr in global memory.
// A bucket is handled by a team of d / 64 lanes (at most a warp, at least one lane), so that the
// sequential walk over a lane's nonzeros is long enough to amortise the team's scans.
#include <mutex>

#include "elias_common.cuh"

namespace qsgd {

namespace {

constexpr int kThreads = 256;
constexpr int kWarps = kThreads / 32;

struct Ctrl {                 // control block at the end of the workspace
  uint64_t total_bits;
  uint64_t payload_bytes;
  uint32_t ok;                // 1 when the message fits out_capacity
  uint32_t arrived;           // CTAs of the length kernel that have published their sum
};

struct Teams {
  uint32_t lpb;               // lanes per bucket (power of two, <= 32)
  uint32_t seg;               // coordinates per lane
  uint32_t nbc;               // buckets per CTA
};

Teams make_teams(uint32_t d) {
  Teams t;
  const bool pow2 = (d & (d - 1)) == 0;
  t.lpb = 32;
  if (pow2) { t.lpb = d / 64; if (t.lpb < 1) t.lpb = 1; if (t.lpb > 32) t.lpb = 32; }
  t.seg = d / t.lpb;
  t.nbc = kWarps * (32 / t.lpb);
  return t;
}

struct EliasWs {
  uint8_t* fixed;             // fixed-width intermediate
  uint32_t* len;              // L_b
  uint32_t* lane_rec;         // per lane of every bucket team: its bits | (previous nonzero + 1) << 16
  uint64_t* cta_sums;         // per scatter CTA: sum of its buckets' lengths, then exclusive prefix
  Ctrl* ctrl;
  size_t bytes;
};

EliasWs carve(uint8_t* ws, uint64_t n, uint32_t d, uint32_t s) {
  const FixedLayout L = make_fixed_layout(n, d, s);
  const Teams tm = make_teams(d);
  EliasWs w;
  size_t o = 0;
  w.fixed = ws + o; o += align16(L.total);
  w.len = reinterpret_cast<uint32_t*>(ws + o); o += align16(4 * L.B);
  w.lane_rec = reinterpret_cast<uint32_t*>(ws + o); o += align16(4 * L.B * tm.lpb);
  const uint64_t ctas = (L.B + tm.nbc - 1) / tm.nbc;
  w.cta_sums = reinterpret_cast<uint64_t*>(ws + o); o += align16(8 * (ctas + 1));
  w.ctrl = reinterpret_cast<Ctrl*>(ws + o); o += align16(sizeof(Ctrl));
  w.bytes = o;
  return w;
}

// Code table indexed by the bit length m of the integer (1 .. 16), kept in shared memory so that
// lanes with different m read it without divergence:
//   bits 0..7 prefix value P(m), bits 8..15 total code length, bit 17 set for m = 1 (whose code is
//   the single bit 0: the generic formula would leave a 1 in bit 1, this bit removes it).
__device__ __forceinline__ void fill_code_table(uint32_t* tab) {
  const uint32_t m = threadIdx.x;
  if (m < 17) {
    uint32_t pv = 0;
    if (m > 8) pv = (3u << 4) | (m - 1u);
    else if (m > 4) pv = (2u << 3) | (m - 1u);
    else if (m > 2) pv = m - 1u;
    const uint32_t len = m <= 1 ? 1u : m + 1u + elias_prefix_len(m);
    tab[m] = pv | (len << 8) | (m == 1 ? (2u << 16) : 0u);
  }
}

__device__ __forceinline__ uint32_t bit_length(uint32_t k) { return 32u - (uint32_t)__clz((int)k); }

// |Elias(k)| from the table.
__device__ __forceinline__ uint32_t tab_len(const uint32_t* tab, uint32_t k) {
  return (tab[bit_length(k)] >> 8) & 0xFFu;
}

// Elias(k), right-aligned; *len receives its length.
__device__ __forceinline__ uint32_t tab_code(const uint32_t* tab, uint32_t k, uint32_t* len) {
  const uint32_t m = bit_length(k);
  const uint32_t e = tab[m];
  *len = (e >> 8) & 0xFFu;
  return ((((e & 0xFFu) << m) | k) << 1) ^ (e >> 16);
}

// Level field c of a bucket whose level fields start at word pointer lwb.
template <int LB>
__device__ __forceinline__ uint32_t level_at(const uint32_t* __restrict__ lwb, uint32_t c) {
  const uint32_t bit = c * LB;
  return (__ldg(lwb + (bit >> 5)) >> (bit & 31)) & ((1u << LB) - 1u);
}

// Bit j of the result is set iff field j of the level word is nonzero (32 / LB fields).
template <int LB>
__device__ __forceinline__ uint32_t nonzero_mask(uint32_t w) {
  if (LB == 1) return w;
  if (LB == 2) {
    uint32_t y = (w | (w >> 1)) & 0x55555555u;
    y = (y | (y >> 1)) & 0x33333333u;
    y = (y | (y >> 2)) & 0x0F0F0F0Fu;
    y = (y | (y >> 4)) & 0x00FF00FFu;
    return (y | (y >> 8)) & 0xFFFFu;
  }
  if (LB == 4) {
    uint32_t y = w | (w >> 1);
    y = (y | (y >> 2)) & 0x11111111u;
    y = (y | (y >> 3)) & 0x03030303u;
    y = (y | (y >> 6)) & 0x000F000Fu;
    return (y | (y >> 12)) & 0xFFu;
  }
  uint32_t y = w | (w >> 4);
  y |= y >> 2;
  y = (y | (y >> 1)) & 0x01010101u;
  y = (y | (y >> 7)) & 0x00030003u;
  return (y | (y >> 14)) & 0xFu;
}

// Walks the nonzero levels of bucket-relative coordinates [c_lo, c_hi) in index order and
// calls visit(position, level). When the range starts on a 32-coordinate boundary (every
// power-of-two bucket size) it is processed in blocks of 64 coordinates: the nonzero fields of a
// block are first condensed into a 64-bit mask, so the visiting loop runs once per nonzero of
// the lane and not once per (word, most loaded lane) pair. Otherwise words are walked one by one.
template <int LB, typename F>
__device__ __forceinline__ void for_each_nonzero(const uint32_t* __restrict__ lwb, uint32_t c_lo,
                                                 uint32_t c_hi, F&& visit) {
  constexpr uint32_t kMask = (1u << LB) - 1u;
  constexpr uint32_t kFields = 32u / LB;           // fields per word
  if ((c_lo & 31u) == 0u) {
    for (uint32_t c0 = c_lo; c0 < c_hi; c0 += 64u) {
      const uint32_t* wp = lwb + ((c0 * LB) >> 5);
      unsigned long long m = 0ull;
#pragma unroll
      for (uint32_t j = 0; j < 2u * LB; ++j) {
        const uint32_t w = (c0 + j * kFields < c_hi) ? __ldg(wp + j) : 0u;
        m |= (unsigned long long)nonzero_mask<LB>(w) << (j * kFields);
      }
      while (m) {
        const uint32_t pos = c0 + (uint32_t)__ffsll((long long)m) - 1u;
        m &= m - 1ull;
        if (pos < c_hi) {
          const uint32_t bit = pos * LB;
          visit(pos, (__ldg(lwb + (bit >> 5)) >> (bit & 31u)) & kMask);
        }
      }
    }
    return;
  }
  uint32_t c = c_lo;
  while (c < c_hi) {
    const uint32_t bit = c * LB;
    const uint32_t sh = bit & 31u;
    uint32_t w = __ldg(lwb + (bit >> 5)) >> sh;
    const uint32_t fields = (32u - sh) / LB;
    const uint32_t cnt = min(fields, c_hi - c);
    if (cnt * LB < 32u) w &= (1u << (cnt * LB)) - 1u;
    while (w) {
      const uint32_t fb = ((uint32_t)__ffs((int)w) - 1u) & ~(uint32_t)(LB - 1);   // first bit of the field
      const uint32_t level = (w >> fb) & kMask;
      visit(c + fb / LB, level);
      w &= ~(kMask << fb);
    }
    c += cnt;
  }
}

struct LaneSummary {
  uint32_t bits;      // bits of this lane's codes, excluding the gap code of its first nonzero
  int32_t first;      // first nonzero position in the lane's range, -1 if none
  int32_t last;       // last nonzero position, -1 if none
};

// Sum over the nonzero fields of one level word of 1 + |Elias(level)| (sign bit and level code),
// without a loop: |Elias(level)| grows by 1, 2, 3, 1, 4, 1, 1, 1 when the level reaches 1, 2, 4, 8,
// 16, 32, 64, 128 (Appendix A.2 lengths 1, 3, 6, 7, 11, 12, 13, 14), so the per-field sum is a weighted
// count of "level >= 2^j" masks, added up across the fields of the word.
template <int LB>
__device__ __forceinline__ uint32_t level_code_bits(uint32_t w) {
  if (LB == 1) return 2u * (uint32_t)__popc(w);
  if (LB == 2) {
    const uint32_t b1 = (w >> 1) & 0x55555555u;
    return 2u * (uint32_t)(__popc(b1 | (w & 0x55555555u)) + __popc(b1));
  }
  if (LB == 4) {
    const uint32_t t3 = w >> 3;
    const uint32_t ge8 = t3 & 0x11111111u;
    const uint32_t ge4 = (t3 | (w >> 2)) & 0x11111111u;
    const uint32_t ge2 = (ge4 | (w >> 1)) & 0x11111111u;
    const uint32_t ge1 = (ge2 | w) & 0x11111111u;
    const uint32_t x = ge8 + 3u * ge4 + 2u * (ge1 + ge2);              // at most 8 per nibble
    const uint32_t y = (x & 0x0F0F0F0Fu) + ((x >> 4) & 0x0F0F0F0Fu);
    return (y * 0x01010101u) >> 24;
  }
  const uint32_t ge128 = (w >> 7) & 0x01010101u;
  const uint32_t ge64 = (ge128 | (w >> 6)) & 0x01010101u;
  const uint32_t ge32 = (ge64 | (w >> 5)) & 0x01010101u;
  const uint32_t ge16 = (ge32 | (w >> 4)) & 0x01010101u;
  const uint32_t ge8 = (ge16 | (w >> 3)) & 0x01010101u;
  const uint32_t ge4 = (ge8 | (w >> 2)) & 0x01010101u;
  const uint32_t ge2 = (ge4 | (w >> 1)) & 0x01010101u;
  const uint32_t ge1 = (ge2 | w) & 0x01010101u;
  const uint32_t x = 2u * (ge1 + ge2) + 3u * ge4 + ge8 + 4u * ge16 + ge32 + ge64 + ge128;   // at most 15 per byte
  return (x * 0x01010101u) >> 24;
}

// Sum of |Elias(gap)| over the set bits of a 64-coordinate block except the lowest, gap = distance to
// the previous set bit, without a loop: P = "some set bit lies 1 .. 2^b - 1 positions below" is built
// by doubling, and the set bits whose gap has bit length b are those in P_b but not in P_(b-1).
__device__ __forceinline__ uint32_t gap_code_bits(unsigned long long m) {
  unsigned long long prev = 0ull, P = m << 1;
  uint32_t bits = (uint32_t)__popcll(m & P);                            // gap 1: code "0"
  prev = P; P = P | (m << 2) | (P << 2);
  bits += 3u * (uint32_t)__popcll(m & P & ~prev);                       // gaps 2 .. 3
  prev = P; P = P | (m << 4) | (P << 4);
  bits += 6u * (uint32_t)__popcll(m & P & ~prev);                       // gaps 4 .. 7
  prev = P; P = P | (m << 8) | (P << 8);
  bits += 7u * (uint32_t)__popcll(m & P & ~prev);                       // gaps 8 .. 15
  prev = P; P = P | (m << 16) | (P << 16);
  bits += 11u * (uint32_t)__popcll(m & P & ~prev);                      // gaps 16 .. 31
  prev = P; P = P | (m << 32) | (P << 32);
  bits += 12u * (uint32_t)__popcll(m & P & ~prev);                      // gaps 32 .. 63
  return bits;
}

// whole_blocks: the lanes' ranges are multiples of 64 coordinates, so every level word this lane
// reads holds only its own coordinates (or, in the last bucket, coordinates past the end of the vector).
template <int LB>
__device__ __forceinline__ LaneSummary summarize_sparse(const uint32_t* tab, const uint32_t* __restrict__ lwb,
                                                        uint32_t c_lo, uint32_t c_hi, bool whole_blocks) {
  LaneSummary s{0u, -1, -1};
  if (whole_blocks) {
    // Blocks of 64 coordinates, no loop over the nonzeros: code lengths come from counting. Fields
    // past the end of the vector are zero in the fixed-width layout, so a ragged c_hi needs no mask
    // beyond not reading words that start past it.
    constexpr uint32_t kFields = 32u / LB;
    for (uint32_t c0 = c_lo; c0 < c_hi; c0 += 64u) {
      const uint32_t* wp = lwb + ((c0 * LB) >> 5);
      unsigned long long m = 0ull;
      uint32_t bits = 0;
#pragma unroll
      for (uint32_t j = 0; j < 2u * LB; ++j) {
        const uint32_t w = (c0 + j * kFields < c_hi) ? __ldg(wp + j) : 0u;
        m |= (unsigned long long)nonzero_mask<LB>(w) << (j * kFields);
        bits += level_code_bits<LB>(w);
      }
      if (m) {
        const int32_t lowest = (int32_t)c0 + __ffsll((long long)m) - 1;
        if (s.first < 0) s.first = lowest;
        else bits += tab_len(tab, (uint32_t)(lowest - s.last));          // gap across two blocks of this lane
        s.last = (int32_t)c0 + 63 - __clzll((long long)m);
        s.bits += bits + gap_code_bits(m);
      }
    }
    return s;
  }
  for_each_nonzero<LB>(lwb, c_lo, c_hi, [&](uint32_t pos, uint32_t level) {
    const bool is_first = s.first < 0;
    const uint32_t gap_bits = tab_len(tab, is_first ? 1u : pos - (uint32_t)s.last);
    s.first = is_first ? (int32_t)pos : s.first;
    s.bits += (is_first ? 0u : gap_bits) + 1u + tab_len(tab, level);
    s.last = (int32_t)pos;
  });
  return s;
}

// whole_blocks as above: whole level words are loaded once and their fields taken from the register
// (fields past the end of the vector are zero in the fixed-width layout but are not coordinates: the
// count stops at c_hi).
template <int LB>
__device__ __forceinline__ uint32_t summarize_dense(const uint32_t* tab, const uint32_t* __restrict__ lwb,
                                                    uint32_t c_lo, uint32_t c_hi, bool whole_blocks) {
  uint32_t bits = 0;
  if (whole_blocks) {
    constexpr uint32_t kFields = 32u / LB, kMask = (1u << LB) - 1u;
    for (uint32_t c0 = c_lo; c0 < c_hi; c0 += 64u) {
      const uint32_t* wp = lwb + ((c0 * LB) >> 5);
#pragma unroll
      for (uint32_t j = 0; j < 2u * LB; ++j) {
        const uint32_t cw = c0 + j * kFields;                 // first coordinate of this word
        if (cw >= c_hi) break;
        const uint32_t w = __ldg(wp + j);
        const uint32_t cnt = min(kFields, c_hi - cw);
        if (cnt == kFields) {
#pragma unroll
          for (uint32_t f = 0; f < kFields; ++f) bits += 1u + tab_len(tab, ((w >> (f * LB)) & kMask) + 1u);
        } else {
          for (uint32_t f = 0; f < cnt; ++f) bits += 1u + tab_len(tab, ((w >> (f * LB)) & kMask) + 1u);
        }
      }
    }
    return bits;
  }
  for (uint32_t c = c_lo; c < c_hi; ++c) bits += 1u + tab_len(tab, level_at<LB>(lwb, c) + 1u);
  return bits;
}

// Position of the last nonzero in the team's lanes before this one (-1 if none).
__device__ __forceinline__ int32_t prev_nonzero_before_lane(int32_t last, uint32_t tl, uint32_t lpb) {
  int32_t run = last;                           // inclusive max-scan of `last` inside the team
#pragma unroll
  for (int o = 1; o < 32; o <<= 1) {
    const int32_t t = __shfl_up_sync(0xffffffffu, run, o, 32);
    if ((uint32_t)o < lpb && tl >= (uint32_t)o) run = max(run, t);
  }
  const int32_t excl = __shfl_up_sync(0xffffffffu, run, 1, 32);
  return tl == 0 ? -1 : excl;
}

struct ScanArgs {              // what the last CTA of the length kernel needs for the scan
  uint64_t ctas;
  size_t out_capacity;
  Ctrl* ctrl;
  uint64_t* out_bits;
  uint32_t* status_dev;
  uint8_t* out;
};

struct BucketParams {
  const float* A;
  const uint32_t* sign;
  const uint32_t* level;
  uint64_t n;
  uint32_t d;
  uint64_t B;
  uint32_t lpb, seg, nbc;
};

// Bits of this lane's part of its bucket's string (the scale's 32 bits go with team lane 0).
template <int LB, bool DENSE>
__device__ __forceinline__ uint32_t lane_bits(const uint32_t* tab, const uint32_t* __restrict__ lwb, uint32_t lpb,
                                              uint32_t c_lo, uint32_t c_hi, uint32_t tl, bool live,
                                              bool whole_blocks, int32_t* prev_out) {
  uint32_t bits = 0;
  int32_t prev = -1;
  if (DENSE) {
    if (live) bits = summarize_dense<LB>(tab, lwb, c_lo, c_hi, whole_blocks);
  } else {
    LaneSummary s{0u, -1, -1};
    if (live) s = summarize_sparse<LB>(tab, lwb, c_lo, c_hi, whole_blocks);
    prev = prev_nonzero_before_lane(s.last, tl, lpb);
    bits = s.bits + (s.first >= 0 ? tab_len(tab, (uint32_t)(s.first - prev)) : 0u);
  }
  if (live && tl == 0) bits += 32u;
  *prev_out = prev;
  return bits;
}

// Sum over the lanes of a team (every lane of the team receives it).
__device__ __forceinline__ uint32_t team_sum(uint32_t v, uint32_t lpb) {
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) {
    const uint32_t t = __shfl_xor_sync(0xffffffffu, v, o);
    if ((uint32_t)o < lpb) v += t;
  }
  return v;
}

// ---- scan of the per-CTA sums, run by the CTA of the length kernel that finishes last ------------
__device__ __forceinline__ uint64_t block_exclusive_scan(uint64_t v, uint64_t* total) {
  __shared__ uint64_t warp_sums[32];
  const uint32_t lane = threadIdx.x & 31, warp = threadIdx.x >> 5, nwarps = blockDim.x >> 5;
  uint64_t inc = v;
#pragma unroll
  for (int o = 1; o < 32; o <<= 1) {
    const uint64_t t = __shfl_up_sync(0xffffffffu, inc, o);
    if (lane >= (uint32_t)o) inc += t;
  }
  if (lane == 31) warp_sums[warp] = inc;
  __syncthreads();
  uint64_t before = 0, all = 0;
  for (uint32_t w = 0; w < nwarps; ++w) {
    const uint64_t t = warp_sums[w];
    if (w < warp) before += t;
    all += t;
  }
  __syncthreads();
  *total = all;
  return before + inc - v;
}

// In place: cta_sums[c] becomes the first payload bit of CTA c's run, cta_sums[ctas] the payload
// length. Also: message geometry, capacity check, and zeroes in every payload word that two
// scatter CTAs share (they OR into those; all other words are stored whole) plus the padding.
// Called by all threads of one CTA.
__device__ __forceinline__ void scan_cta_sums(uint64_t* cta_sums, uint64_t ctas, uint64_t B, size_t out_capacity,
                                              Ctrl* ctrl, uint64_t* out_bits, uint32_t* status_dev, uint8_t* out) {
  __shared__ uint32_t ok_s;
  __shared__ uint64_t pay_s;
  // every thread owns a contiguous chunk of the sums: one block-wide scan in total
  const uint64_t chunk = (ctas + blockDim.x - 1) / blockDim.x;
  const uint64_t lo = min((uint64_t)threadIdx.x * chunk, ctas), hi = min(lo + chunk, ctas);
  uint64_t mine = 0;
#pragma unroll 8
  for (uint64_t i = lo; i < hi; ++i) mine += __ldcg(cta_sums + i);
  uint64_t total;
  uint64_t run = block_exclusive_scan(mine, &total);
  if (threadIdx.x == 0) {
    const uint64_t pay = align16((total + 7) / 8);
    const uint64_t total_bytes = pay + 8 * (B + 1);
    const bool ok = total_bytes <= out_capacity;
    ctrl->total_bits = total;
    ctrl->payload_bytes = pay;
    ctrl->ok = ok ? 1u : 0u;
    out_bits[0] = total; out_bits[1] = pay; out_bits[2] = total_bytes; out_bits[3] = 0;
    if (!ok) atomicOr(status_dev, QSGD_DEV_CAPACITY);
    ok_s = ok ? 1u : 0u;
    pay_s = pay;
    cta_sums[ctas] = total;
  }
  __syncthreads();
  const bool ok = ok_s != 0;
  uint32_t* words = reinterpret_cast<uint32_t*>(out);
#pragma unroll 8
  for (uint64_t i = lo; i < hi; ++i) {
    const uint64_t v = __ldcg(cta_sums + i);
    cta_sums[i] = run;
    if (ok && (run & 31)) words[run >> 5] = 0u;
    run += v;
  }
  if (ok && threadIdx.x == 0)
    for (uint64_t w = total >> 5; w < pay_s / 4; ++w) words[w] = 0u;        // tail word + padding
}

// ---- 2. string length per bucket, sum per CTA ------------------------------------------------------
template <int LB, bool DENSE>
__global__ void __launch_bounds__(kThreads) elias_length_kernel(const BucketParams p,
                                                                uint32_t* __restrict__ len,
                                                                uint32_t* __restrict__ lane_rec,
                                                                uint64_t* cta_sums, const ScanArgs sa) {
  __shared__ uint32_t warp_sum[kWarps];
  __shared__ uint32_t is_last;
  __shared__ uint32_t tab[17];
  fill_code_table(tab);
  __syncthreads();
  chain_wait();                                    // the fields come from the kernel ahead
  const uint32_t lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  const uint32_t tl = lane & (p.lpb - 1), team = lane / p.lpb, bpw = 32 / p.lpb;
  const uint64_t b = (uint64_t)blockIdx.x * p.nbc + warp * bpw + team;
  const bool live = b < p.B;
  const uint64_t base = live ? b * p.d : 0;
  const uint32_t db = live ? (uint32_t)min((uint64_t)p.d, p.n - base) : 0;
  const uint32_t c_lo = min(tl * p.seg, db), c_hi = min(c_lo + p.seg, db);
  const uint32_t* lwb = p.level + ((base * LB) >> 5);            // the bucket's first level word
  int32_t prev;
  const uint32_t bits = lane_bits<LB, DENSE>(tab, lwb, p.lpb, c_lo, c_hi, tl, live, (p.seg & 63u) == 0u, &prev);
  if (live) lane_rec[b * p.lpb + tl] = bits | ((uint32_t)(prev + 1) << 16);   // reused by the scatter
  const uint32_t L = team_sum(bits, p.lpb);
  if (live && tl == 0) len[b] = L;
  uint32_t w = (tl == 0) ? L : 0u;                 // one contribution per bucket
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) w += __shfl_xor_sync(0xffffffffu, w, o);
  if (lane == 0) warp_sum[warp] = w;
  __syncthreads();
  if (threadIdx.x == 0) {
    uint64_t s = 0;
#pragma unroll
    for (int i = 0; i < kWarps; ++i) s += warp_sum[i];
    cta_sums[blockIdx.x] = s;
    // publish, then take a ticket: whoever draws the last one sees every CTA's sum
    __threadfence();
    is_last = atomicAdd(&sa.ctrl->arrived, 1u) == gridDim.x - 1u ? 1u : 0u;
  }
  __syncthreads();
  if (is_last) {
    __threadfence();
    scan_cta_sums(cta_sums, sa.ctas, p.B, sa.out_capacity, sa.ctrl, sa.out_bits, sa.status_dev, sa.out);
  }
}

// ---- 4. scatter ----------------------------------------------------------------------------------
// Lane-private writer into the CTA's staging words in shared memory.
struct StageWriter {
  uint32_t* words;
  uint32_t widx;
  uint64_t buf;
  uint32_t nbuf;
  __device__ __forceinline__ void begin(uint32_t* w, uint32_t start_bit) {
    words = w; widx = start_bit >> 5; buf = 0; nbuf = start_bit & 31;
  }
  __device__ __forceinline__ void put(uint32_t code, uint32_t len) {   // len in [1, 32]
    buf |= (uint64_t)code << (64 - nbuf - len);
    nbuf += len;
    if (nbuf >= 32) {
      atomicOr(words + widx, (uint32_t)(buf >> 32));
      ++widx; buf <<= 32; nbuf -= 32;
    }
  }
  __device__ __forceinline__ void finish() {
    if (nbuf) atomicOr(words + widx, (uint32_t)(buf >> 32));
  }
};

template <int LB, bool DENSE>
__global__ void __launch_bounds__(kThreads) elias_scatter_kernel(const BucketParams p,
                                                                 const uint32_t* __restrict__ len,
                                                                 const uint32_t* __restrict__ lane_rec,
                                                                 const uint64_t* __restrict__ cta_start,
                                                                 const Ctrl* __restrict__ ctrl,
                                                                 uint8_t* __restrict__ out) {
  extern __shared__ uint32_t stage[];
  __shared__ uint32_t warp_sum[kWarps];
  __shared__ uint32_t tab[17];
  // whole code words (code | length << 16) of the integers met most: every level, and gaps below 64
  __shared__ uint32_t level_code[1u << LB];
  __shared__ uint32_t gap_code[64];
  fill_code_table(tab);
  if (!DENSE) {
    for (uint32_t k = threadIdx.x; k < (1u << LB) + 64u; k += kThreads) {
      const uint32_t v = k < (1u << LB) ? k : k - (1u << LB);
      uint32_t ln = 0;
      const uint32_t code = v ? elias_code(v, &ln) : 0u;
      (k < (1u << LB) ? level_code[v] : gap_code[v]) = code | (ln << 16);
    }
  }
  chain_wait();                                    // ctrl, lengths and sums come from the kernel ahead
  if (!ctrl->ok) return;
  const uint32_t lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  const uint32_t tl = lane & (p.lpb - 1), team = lane / p.lpb, bpw = 32 / p.lpb;
  const uint64_t b = (uint64_t)blockIdx.x * p.nbc + warp * bpw + team;
  const bool live = b < p.B;
  const uint64_t base = live ? b * p.d : 0;
  const uint32_t db = live ? (uint32_t)min((uint64_t)p.d, p.n - base) : 0;
  const uint32_t c_lo = min(tl * p.seg, db), c_hi = min(c_lo + p.seg, db);

  const uint64_t start = __ldg(cta_start + blockIdx.x), stop = __ldg(cta_start + blockIdx.x + 1);
  const uint32_t lead = (uint32_t)(start & 31);                     // bits of the first word owned by the previous CTA
  const uint32_t span = (uint32_t)(stop - start);                   // bits of this CTA's run
  const uint32_t nwords = (lead + span + 31) >> 5;
  for (uint32_t j = threadIdx.x; j < nwords; j += kThreads) stage[j] = 0u;

  // bit offset of every bucket inside the CTA's run: scan of the bucket lengths
  const uint32_t L = (live && tl == 0) ? __ldg(len + b) : 0u;
  uint32_t inc = L;
#pragma unroll
  for (int o = 1; o < 32; o <<= 1) {
    const uint32_t t = __shfl_up_sync(0xffffffffu, inc, o);
    if (lane >= (uint32_t)o) inc += t;
  }
  if (lane == 31) warp_sum[warp] = inc;
  __syncthreads();                                                  // staging zeroed, warp sums visible
  uint32_t before = 0;
#pragma unroll
  for (int w = 0; w < kWarps; ++w) if ((uint32_t)w < warp) before += warp_sum[w];
  uint32_t bucket_off = before + inc - L;                           // valid in team lane 0
  bucket_off = __shfl_sync(0xffffffffu, bucket_off, (int)(lane - tl));
  const uint32_t Lb = __shfl_sync(0xffffffffu, L, (int)(lane - tl));
  if (live && tl == 0) {
    uint64_t* table = reinterpret_cast<uint64_t*>(out + ctrl->payload_bytes);
    table[b] = start + bucket_off;
    if (b == p.B - 1) table[p.B] = start + bucket_off + Lb;
  }

  // this lane's first bit inside its bucket: scan of the lane lengths over the team
  int32_t prev;
  const uint32_t* lwb = p.level + ((base * LB) >> 5);            // the bucket's first level word
  const uint32_t* swb = p.sign + (base >> 5);                    // ... and first sign word
  // this lane's share of the string and the nonzero before it were counted by the length kernel
  const uint32_t rec = live ? __ldg(lane_rec + b * p.lpb + tl) : 0u;
  const uint32_t bits = rec & 0xFFFFu;
  prev = (int32_t)(rec >> 16) - 1;
  uint32_t linc = bits;
#pragma unroll
  for (int o = 1; o < 32; o <<= 1) {
    const uint32_t t = __shfl_up_sync(0xffffffffu, linc, o);
    if ((uint32_t)o < p.lpb && tl >= (uint32_t)o) linc += t;
  }
  if (bits != 0) {
    StageWriter bw;
    bw.begin(stage, lead + bucket_off + (linc - bits));
    if (tl == 0) bw.put(__float_as_uint(__ldg(p.A + b)), 32);
    if (DENSE && (p.seg & 63u) == 0u) {
      // ranges of whole 64-coordinate blocks: sign and level words are loaded once per block and word
      constexpr uint32_t kFields = 32u / LB, kMask = (1u << LB) - 1u;
      for (uint32_t c0 = c_lo; c0 < c_hi; c0 += 64u) {
        const uint32_t* wp = lwb + ((c0 * LB) >> 5);
        const uint32_t s0 = __ldg(swb + (c0 >> 5)), s1 = (c0 + 32u < c_hi) ? __ldg(swb + (c0 >> 5) + 1) : 0u;
        const unsigned long long signs = (unsigned long long)s0 | ((unsigned long long)s1 << 32);
#pragma unroll
        for (uint32_t j = 0; j < 2u * LB; ++j) {
          const uint32_t off = j * kFields;                   // first coordinate of this word in the block
          if (c0 + off >= c_hi) break;
          const uint32_t w = __ldg(wp + j);
          const uint32_t cnt = min(kFields, c_hi - (c0 + off));
          for (uint32_t f = 0; f < cnt; ++f) {
            uint32_t ln;
            const uint32_t code = tab_code(tab, ((w >> (f * LB)) & kMask) + 1u, &ln);
            bw.put((((uint32_t)(signs >> (off + f)) & 1u) << ln) | code, ln + 1);
          }
        }
      }
    } else if (DENSE) {
      for (uint32_t c = c_lo; c < c_hi; ++c) {
        const uint32_t sg = (__ldg(swb + (c >> 5)) >> (c & 31)) & 1u;
        uint32_t ln;
        const uint32_t code = tab_code(tab, level_at<LB>(lwb, c) + 1u, &ln);
        bw.put((sg << ln) | code, ln + 1);
      }
    } else if ((p.seg & 63u) == 0u) {
      // Ranges of whole 64-coordinate blocks (every power-of-two d >= 64): the block's nonzero mask
      // and sign bits sit in registers, code words come whole from the two tables.
      constexpr uint32_t kFields = 32u / LB, kMask = (1u << LB) - 1u;
      for (uint32_t c0 = c_lo; c0 < c_hi; c0 += 64u) {
        const uint32_t* wp = lwb + ((c0 * LB) >> 5);
        unsigned long long m = 0ull;
#pragma unroll
        for (uint32_t j = 0; j < 2u * LB; ++j) {
          const uint32_t w = (c0 + j * kFields < c_hi) ? __ldg(wp + j) : 0u;
          m |= (unsigned long long)nonzero_mask<LB>(w) << (j * kFields);
        }
        const uint32_t s0 = __ldg(swb + (c0 >> 5)), s1 = (c0 + 32u < c_hi) ? __ldg(swb + (c0 >> 5) + 1) : 0u;
        const unsigned long long signs = (unsigned long long)s0 | ((unsigned long long)s1 << 32);
        while (m) {
          const uint32_t off = (uint32_t)__ffsll((long long)m) - 1u;
          m &= m - 1ull;
          const uint32_t pos = c0 + off, bit = off * LB;
          const uint32_t level = (__ldg(wp + (bit >> 5)) >> (bit & 31u)) & kMask;
          const uint32_t gap = pos - (uint32_t)prev;
          uint32_t gcode, gl;
          if (gap < 64u) {
            const uint32_t e = gap_code[gap];
            gcode = e & 0xFFFFu;
            gl = e >> 16;
          } else {
            gcode = tab_code(tab, gap, &gl);
          }
          const uint32_t e = level_code[level];
          const uint32_t ll = e >> 16;
          const uint32_t lcode = (e & 0xFFFFu) | ((uint32_t)((signs >> off) & 1ull) << ll);
          if (gl + ll + 1u <= 32u) {                     // gap, sign and level in one piece (the rule)
            bw.put((gcode << (ll + 1u)) | lcode, gl + ll + 1u);
          } else {
            bw.put(gcode, gl);
            bw.put(lcode, ll + 1u);
          }
          prev = (int32_t)pos;
        }
      }
    } else {
      for_each_nonzero<LB>(lwb, c_lo, c_hi, [&](uint32_t pos, uint32_t level) {
        uint32_t gl, ll;
        const uint32_t gcode = tab_code(tab, pos - (uint32_t)prev, &gl);
        const uint32_t sg = (__ldg(swb + (pos >> 5)) >> (pos & 31)) & 1u;
        uint32_t lcode = tab_code(tab, level, &ll);
        lcode |= sg << ll;
        if (gl + ll + 1u <= 32u) {                     // gap, sign and level in one piece (the rule)
          bw.put((gcode << (ll + 1u)) | lcode, gl + ll + 1u);
        } else {
          bw.put(gcode, gl);
          bw.put(lcode, ll + 1u);
        }
        prev = (int32_t)pos;
      });
    }
    bw.finish();
  }
  __syncthreads();
  // flush: whole words are stored; the first / last word may be shared with the neighbouring CTA
  uint32_t* gw = reinterpret_cast<uint32_t*>(out) + (start >> 5);
  const bool last_shared = ((lead + span) & 31) != 0;
  for (uint32_t j = threadIdx.x; j < nwords; j += kThreads) {
    const uint32_t v = stage[j];
    const bool shared = (j == 0 && lead != 0) || (j == nwords - 1 && last_shared);
    if (shared) atomicOr(gw + j, v);
    else gw[j] = v;
  }
}

uint32_t host_elias_len(uint32_t k) {
  uint32_t len = 1;
  while (k > 1) {
    uint32_t m = 0;
    for (uint32_t t = k; t; t >>= 1) ++m;
    len += m;
    k = m - 1;
  }
  return len;
}

template <int LB, bool DENSE>
int run_pipeline(BucketParams& bp, const EliasWs& w, uint32_t s, uint8_t* out, size_t out_capacity,
                 uint64_t* out_bits, uint32_t* status_dev, cudaStream_t stream) {
  const Teams tm = make_teams(bp.d);
  bp.lpb = tm.lpb; bp.seg = tm.seg; bp.nbc = tm.nbc;
  const uint64_t ctas = (bp.B + tm.nbc - 1) / tm.nbc;
  {
    ScanArgs sa;
    sa.ctas = ctas; sa.out_capacity = out_capacity; sa.ctrl = w.ctrl; sa.out_bits = out_bits;
    sa.status_dev = status_dev; sa.out = out;
    ScopedKernel sk(kKernEliasLength, stream);
    const cudaError_t e = launch_chained(elias_length_kernel<LB, DENSE>, (uint32_t)ctas, kThreads, 0, stream, bp, w.len,
                                         w.lane_rec, w.cta_sums, sa);
    if (e != cudaSuccess) return (int)e;
  }
  {
    // staging: the longest legal strings of a CTA's buckets, plus the shared lead-in word
    const uint32_t per = DENSE ? 1 + host_elias_len(s + 1) : 2 + host_elias_len(s);
    const size_t run_bits = (size_t)tm.nbc * (32 + (size_t)bp.d * per);
    const size_t smem = ((run_bits + 31) / 32 + 4) * 4;
    auto kern = elias_scatter_kernel<LB, DENSE>;
    if (smem > 48 * 1024) {
      cudaError_t e = cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
      if (e != cudaSuccess) return (int)e;
    }
    ScopedKernel sk(kKernEliasScatter, stream);
    return (int)launch_chained(kern, (uint32_t)ctas, kThreads, smem, stream, bp, w.len, w.lane_rec, w.cta_sums, w.ctrl, out);
  }
}

}  // namespace

size_t elias_workspace_bytes(uint64_t n, uint32_t d, uint32_t s) {
  return carve(nullptr, n, d, s).bytes;
}

int launch_elias_encode(const float* g, uint64_t n, uint32_t d, uint32_t s, int norm_kind,
                        bool dense, uint64_t seed, uint32_t step, uint32_t worker, uint8_t* out,
                        size_t out_capacity, uint64_t* out_bits, uint8_t* workspace,
                        uint32_t* status_dev, const BucketMap& map, cudaStream_t stream) {
  const EliasWs w = carve(workspace, n, d, s);
  int st = launch_quantize_fixed(g, n, d, s, norm_kind, seed, step, worker, w.fixed, status_dev, nullptr,
                                 &w.ctrl->arrived, map, stream);
  if (st) return st;
  const FixedLayout L = make_fixed_layout(n, d, s);
  BucketParams bp;
  bp.A = reinterpret_cast<const float*>(w.fixed);
  bp.sign = reinterpret_cast<const uint32_t*>(w.fixed + L.off_sign);
  bp.level = reinterpret_cast<const uint32_t*>(w.fixed + L.off_level);
  bp.n = n; bp.d = d; bp.B = L.B;
#define QSGD_RUN(LBV)                                                                            \
  (dense ? run_pipeline<LBV, true>(bp, w, s, out, out_capacity, out_bits, status_dev, stream)       \
         : run_pipeline<LBV, false>(bp, w, s, out, out_capacity, out_bits, status_dev, stream))
  switch (L.lb) {
    case 1: return QSGD_RUN(1);
    case 2: return QSGD_RUN(2);
    case 4: return QSGD_RUN(4);
    default: return QSGD_RUN(8);
  }
#undef QSGD_RUN
}

}  // namespace qsgd

// ================================================================================================
// Elias encode with library-owned scratch (see qsgd_encode_elias_static in include/qsgd.h).
//
// The scratch lives in this translation unit as one file-scope device array, so the entry point
// never asks the driver (or anybody's allocator) for memory. In host code the name of a
// __device__ array is only a handle for the runtime: its device address has to be looked up with
// cudaGetSymbolAddress, once per device, with that device current. The looked-up pointer is what
// the kernels receive.
// ================================================================================================
namespace qsgd {
namespace {

constexpr size_t kStaticScratchBytes = (size_t)QSGD_STATIC_SCRATCH_BYTES;
static __device__ __align__(256) unsigned char g_static_scratch[kStaticScratchBytes];

constexpr int kMaxDevices = 64;
static std::mutex g_scratch_mu;
static uint8_t* g_scratch_ptr[kMaxDevices] = {};

// Device address of the scratch array on the current device; looked up on first use.
int static_scratch_pointer(uint8_t** out) {
  int dev = -1;
  cudaError_t e = cudaGetDevice(&dev);
  if (e != cudaSuccess) return (int)e;
  if (dev < 0 || dev >= kMaxDevices) return (int)cudaErrorInvalidDevice;
  std::lock_guard<std::mutex> lk(g_scratch_mu);
  if (!g_scratch_ptr[dev]) {
    void* p = nullptr;
    e = cudaGetSymbolAddress(&p, g_static_scratch);
    if (e != cudaSuccess) return (int)e;
    if (!p) return (int)cudaErrorInvalidSymbol;
    g_scratch_ptr[dev] = static_cast<uint8_t*>(p);
  }
  *out = g_scratch_ptr[dev];
  return 0;
}

}  // namespace
}  // namespace qsgd

extern "C" {

size_t qsgd_static_scratch_bytes(void) { return qsgd::kStaticScratchBytes; }

int qsgd_encode_elias_static(const float* g, uint64_t n, uint32_t bucket, uint32_t s, int norm_kind,
                             int code_kind, uint64_t seed, uint32_t step, uint32_t worker, void* out,
                             size_t out_capacity, uint64_t* out_bits, uint32_t* status_dev,
                             qsgd_stream_t stream) {
  using namespace qsgd;
  if (!g || !out || !out_bits || !status_dev) return QSGD_ERR_NULL;
  if (n == 0 || n > QSGD_MAX_COORDS) return QSGD_ERR_SIZE;
  if (bucket < 32 || bucket > QSGD_MAX_BUCKET || (bucket & 31u)) return QSGD_ERR_BUCKET;
  if (s < 1 || s > QSGD_MAX_LEVELS) return QSGD_ERR_LEVELS;
  if (code_kind != QSGD_CODE_ELIAS && code_kind != QSGD_CODE_ELIAS_DENSE) return QSGD_ERR_KIND;
  if (norm_kind != QSGD_NORM_L2 && norm_kind != QSGD_NORM_MAX) return QSGD_ERR_KIND;
  if ((reinterpret_cast<uintptr_t>(g) & 15u) || (reinterpret_cast<uintptr_t>(out) & 15u)) return QSGD_ERR_ALIGN;
  const uint64_t B = (n + bucket - 1) / bucket;
  if (out_capacity < align16(4 * B) + 8 * (B + 1)) return QSGD_ERR_CAPACITY;
  if (elias_workspace_bytes(n, bucket, s) > kStaticScratchBytes) return QSGD_ERR_SCRATCH;
  uint8_t* scratch = nullptr;
  const int st = static_scratch_pointer(&scratch);
  if (st) return st;
  return launch_elias_encode(g, n, bucket, s, norm_kind, code_kind == QSGD_CODE_ELIAS_DENSE, seed, step,
                             worker, static_cast<uint8_t*>(out), out_capacity, out_bits, scratch,
                             status_dev, no_map(), static_cast<cudaStream_t>(stream));
}

}  // extern "C"
