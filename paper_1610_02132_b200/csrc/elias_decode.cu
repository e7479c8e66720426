// Decode-and-aggregate, Elias path, optionally fused with the SGD step (Section 3.1: "read off
// 32 bits to construct the norm, then iteratively ... read off the positions and values of the
// nonzeros"; Appendix A.2 decoder; Algorithm 1 for the sum and the step).
//
// A string S can only be parsed front to back, but buckets and peers are independent once the
// per-bucket offset table gives each string's first bit. A warp owns a group of G buckets.
// Phase 1 (parse): lane (g, k) reads peer k's string of bucket g through a 64-bit register
// window (next word prefetched) and rebuilds that peer's *fixed-width fields* -- level fields
// and sign bitmap -- for the bucket in shared memory. Phase 2 (apply): exactly the fixed-width
// decoder's inner loop, reading the fields from shared memory: every lane takes 16 coordinates
// and adds the peers in ascending k, which fixes the summation order however phase 1 was
// scheduled. A slower kernel with byte codes covers shapes whose fields do not fit in shared
// memory.
#include "decode_common.cuh"
#include "elias_common.cuh"

namespace qsgd {

namespace {

constexpr int kWarps = 4;
constexpr int kThreads = kWarps * 32;

struct EliasDecodeParams {
  PeerSet peers;
  uint32_t K;
  uint32_t Kc;         // peers per pass (scratch holds Kc x d codes)
  uint64_t n;
  uint32_t d;
  uint32_t s;
  uint64_t B;
  float* out;          // acc (overwritten) or x (updated in place)
  float c;             // eta / K
  uint32_t* status;
  uint32_t warp_bytes; // shared memory per warp
};

template <typename CodeT> struct CodeTraits;
template <> struct CodeTraits<uint8_t> { static constexpr uint32_t kSignBit = 0x80u; };
template <> struct CodeTraits<uint16_t> { static constexpr uint32_t kSignBit = 0x8000u; };

// Parses one bucket string of one peer into codes[0..db). Returns a QSGD_DEV_* mask.
template <typename CodeT, bool DENSE>
__device__ __forceinline__ uint32_t parse_bucket(const uint32_t* __restrict__ words,
                                                 const uint64_t* __restrict__ table, uint64_t b,
                                                 uint64_t B, uint32_t db, uint32_t s,
                                                 CodeT* __restrict__ codes, float* A_out) {
  const uint64_t lo = __ldg(table + b), hi = __ldg(table + b + 1), all = __ldg(table + B);
  *A_out = 0.f;
  if (hi < lo || hi - lo < 32 || hi > all) return QSGD_DEV_TABLE;
  // the table sits directly behind the payload: its address bounds the payload length
  const uint64_t cap_bits = (uint64_t)((const uint8_t*)table - (const uint8_t*)words) * 8ull;
  if ((const uint8_t*)table > (const uint8_t*)words && all > cap_bits) return QSGD_DEV_TABLE;
  uint64_t pos = lo;
  *A_out = __uint_as_float(peek32(words, pos));
  pos += 32;
  if (DENSE) {
    for (uint32_t c = 0; c < db; ++c) {
      if (pos >= hi) return QSGD_DEV_OVERRUN;
      const uint32_t sg = peek32(words, pos) >> 31;
      pos += 1;
      uint32_t v;
      if (!elias_read(words, pos, v) || pos > hi) return QSGD_DEV_OVERRUN;
      if (v - 1u > s) return QSGD_DEV_LEVEL;
      codes[c] = (CodeT)((v - 1u) | (sg && v > 1u ? CodeTraits<CodeT>::kSignBit : 0u));
    }
    return pos == hi ? 0u : QSGD_DEV_OVERRUN;
  }
  int64_t at = -1;
  while (pos < hi) {
    uint32_t gap, level;
    if (!elias_read(words, pos, gap) || pos >= hi) return QSGD_DEV_OVERRUN;
    at += gap;
    if (at >= (int64_t)db) return QSGD_DEV_POSITION;
    const uint32_t sg = peek32(words, pos) >> 31;
    pos += 1;
    if (!elias_read(words, pos, level) || pos > hi) return QSGD_DEV_OVERRUN;
    if (level < 1u || level > s) return QSGD_DEV_LEVEL;
    codes[at] = (CodeT)(level | (sg ? CodeTraits<CodeT>::kSignBit : 0u));
  }
  return 0u;
}

template <typename CodeT, bool DENSE, bool FUSED>
__global__ void __launch_bounds__(kThreads) decode_elias_slow_kernel(const __grid_constant__ EliasDecodeParams p) {
  extern __shared__ __align__(16) uint8_t smem[];
  __shared__ float xi[256];
  const float sf = (float)p.s;
  for (uint32_t l = threadIdx.x; l < 256; l += kThreads) xi[l] = __fdiv_rn((float)l, sf);
  __syncthreads();

  const uint32_t lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  uint8_t* mine = smem + (size_t)warp * p.warp_bytes;
  float* acc = reinterpret_cast<float*>(mine);                       // d floats
  float* sA = acc + p.d;                                             // Kc floats (padded to 64)
  CodeT* codes = reinterpret_cast<CodeT*>(sA + 64);                  // Kc x d codes
  constexpr uint32_t kSign = CodeTraits<CodeT>::kSignBit;
  constexpr uint32_t kPer16 = 16 / sizeof(CodeT);

  for (uint64_t b = (uint64_t)blockIdx.x * kWarps + warp; b < p.B; b += (uint64_t)gridDim.x * kWarps) {
    const uint64_t base = b * p.d;
    const uint32_t db = (uint32_t)min((uint64_t)p.d, p.n - base);
    for (uint32_t c = lane * 4; c < p.d; c += 128)
      *reinterpret_cast<float4*>(acc + c) = make_float4(0.f, 0.f, 0.f, 0.f);

    for (uint32_t k0 = 0; k0 < p.K; k0 += p.Kc) {
      const uint32_t kc = min(p.Kc, p.K - k0);
      // zero the scratch of this pass
      const uint32_t quads = kc * p.d / kPer16;
      for (uint32_t q = lane; q < quads; q += 32)
        reinterpret_cast<uint4*>(codes)[q] = make_uint4(0u, 0u, 0u, 0u);
      __syncwarp();
      // phase 1: one lane per peer
      for (uint32_t kk = lane; kk < kc; kk += 32) {
        float A;
        const uint32_t st = parse_bucket<CodeT, DENSE>(p.peers.payload[k0 + kk], p.peers.table[k0 + kk],
                                                       b, p.B, db, p.s, codes + (size_t)kk * p.d, &A);
        sA[kk] = A;
        if (st) atomicOr(p.status, st);
      }
      __syncwarp();
      // phase 2: ascending-k sum, 4 coordinates per lane
      for (uint32_t c = lane * 4; c < p.d; c += 128) {
        float4 a = *reinterpret_cast<const float4*>(acc + c);
        for (uint32_t kk = 0; kk < kc; ++kk) {
          uint32_t e[4];
          if (sizeof(CodeT) == 1) {
            const uint32_t w = *reinterpret_cast<const uint32_t*>(codes + (size_t)kk * p.d + c);
            if (w == 0u) continue;
            e[0] = w & 0xFFu; e[1] = (w >> 8) & 0xFFu; e[2] = (w >> 16) & 0xFFu; e[3] = w >> 24;
          } else {
            const uint2 w = *reinterpret_cast<const uint2*>(codes + (size_t)kk * p.d + c);
            if ((w.x | w.y) == 0u) continue;
            e[0] = w.x & 0xFFFFu; e[1] = w.x >> 16; e[2] = w.y & 0xFFFFu; e[3] = w.y >> 16;
          }
          const float A = sA[kk];
          float m[4];
#pragma unroll
          for (int j = 0; j < 4; ++j) {
            const float t = __fmul_rn(A, xi[e[j] & (kSign - 1u)]);
            m[j] = (e[j] & kSign) ? -t : t;
          }
          if (e[0]) a.x = __fadd_rn(a.x, m[0]);
          if (e[1]) a.y = __fadd_rn(a.y, m[1]);
          if (e[2]) a.z = __fadd_rn(a.z, m[2]);
          if (e[3]) a.w = __fadd_rn(a.w, m[3]);
        }
        *reinterpret_cast<float4*>(acc + c) = a;
      }
      __syncwarp();
    }

    // write the bucket: acc, or the SGD step on x
    for (uint32_t c = lane * 4; c < db; c += 128) {
      const float4 a = *reinterpret_cast<const float4*>(acc + c);
      float* o = p.out + base + c;
      if (c + 4 <= db) {
        float4 r = a;
        if (FUSED) {
          const float4 x = *reinterpret_cast<const float4*>(o);
          r.x = __fsub_rn(x.x, __fmul_rn(p.c, a.x)); r.y = __fsub_rn(x.y, __fmul_rn(p.c, a.y));
          r.z = __fsub_rn(x.z, __fmul_rn(p.c, a.z)); r.w = __fsub_rn(x.w, __fmul_rn(p.c, a.w));
        }
        *reinterpret_cast<float4*>(o) = r;
      } else {
        const float t[4] = {a.x, a.y, a.z, a.w};
        for (uint32_t j = 0; c + j < db; ++j) o[j] = FUSED ? __fsub_rn(o[j], __fmul_rn(p.c, t[j])) : t[j];
      }
    }
    __syncwarp();
  }
}

template <typename CodeT, bool DENSE>
int launch_slow(EliasDecodeParams& p, bool fused, cudaStream_t stream) {
  // shared memory per warp: d floats of acc, 64 floats of scales, Kc x d codes
  int dev = 0, max_smem = 0, sms = 0;
  cudaGetDevice(&dev);
  cudaDeviceGetAttribute(&max_smem, cudaDevAttrMaxSharedMemoryPerBlockOptin, dev);
  cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev);
  const size_t fixed = (size_t)p.d * 4 + 64 * 4;
  const size_t budget = ((size_t)max_smem - 2048) / kWarps;
  size_t kc = p.K;
  while (kc > 1 && fixed + kc * p.d * sizeof(CodeT) > budget) kc = (kc + 1) / 2;
  if (fixed + kc * p.d * sizeof(CodeT) > budget) return (int)cudaErrorInvalidConfiguration;
  p.Kc = (uint32_t)kc;
  p.warp_bytes = (uint32_t)align16(fixed + kc * p.d * sizeof(CodeT));
  const size_t smem = (size_t)p.warp_bytes * kWarps;
  auto kern = fused ? decode_elias_slow_kernel<CodeT, DENSE, true> : decode_elias_slow_kernel<CodeT, DENSE, false>;
  cudaError_t e = cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
  if (e != cudaSuccess) return (int)e;
  const uint64_t want = (p.B + kWarps - 1) / kWarps;
  const uint64_t cap = (uint64_t)sms * 16;
  const uint32_t grid = (uint32_t)(want < cap ? want : cap);
  {
    ScopedKernel sk(kKernDecodeElias, stream);
    kern<<<grid, kThreads, smem, stream>>>(p);
  }
  return (int)cudaGetLastError();
}


// ------------------------------------------------------------------------------------------------
// Field-rebuilding decoder
// ------------------------------------------------------------------------------------------------
struct FieldParams {
  PeerSet peers;
  uint32_t K;
  uint32_t Kpad;        // lanes per bucket in the parse phase (power of two, <= 32)
  uint32_t G;           // buckets per warp
  uint64_t n;
  uint32_t d;
  uint32_t s;
  uint64_t B;
  float* out;
  float c;
  uint32_t* status;
  uint32_t row_words;   // per peer row: d * lb / 32 level words, then d / 32 sign words (padded to 4)
  uint32_t bucket_words;  // K rows + K scales, padded to 4
};

// Bit source over the payload: a 64-bit left-aligned window held as two 32-bit halves (all
// shifts are single funnel-shift instructions), with the next payload word prefetched.
struct BitSrc {
  const uint32_t* wp;   // payload word the window started in
  uint32_t idx;         // index (from wp) of `nextw`
  uint32_t nextw;
  uint32_t hi, lo;      // window, most significant bit first
  uint32_t avail;       // valid bits in the window
  __device__ __forceinline__ void open(const uint32_t* words, uint64_t bit) {
    wp = words + (bit >> 5);
    const uint32_t w0 = __ldg(wp), w1 = __ldg(wp + 1);
    nextw = __ldg(wp + 2);
    idx = 2;
    const uint32_t sh = (uint32_t)(bit & 31);
    hi = __funnelshift_l(w1, w0, sh);
    lo = w1 << sh;
    avail = 64 - sh;
  }
  __device__ __forceinline__ void refill() {          // afterwards at least 33 valid bits
    if (avail <= 32) {
      const uint32_t s = 32 - avail;                  // the new word lands s bits above bit 0
      hi |= __funnelshift_lc(nextw, 0u, s);
      lo = __funnelshift_lc(0u, nextw, s);
      avail += 32;
      ++idx;
      nextw = __ldg(wp + idx);
    }
  }
  __device__ __forceinline__ void drop(uint32_t nb) {  // nb in [1, 32]
    hi = __funnelshift_lc(lo, hi, nb);
    lo = __funnelshift_lc(0u, lo, nb);
    avail -= nb;
  }
  __device__ __forceinline__ uint32_t take(uint32_t nb) {   // nb in [1, 32]
    const uint32_t v = hi >> (32 - nb);
    drop(nb);
    return v;
  }
  // Definition A.1 decoder on the window; at most three groups (values < 2^16).
  __device__ __forceinline__ bool elias(uint32_t& value, uint32_t& used) {
    uint32_t N = 1;
#pragma unroll
    for (int it = 0; it < 3; ++it) {
      if ((int32_t)hi >= 0) break;
      const uint32_t nb = N + 1;
      N = take(nb);
      used += nb;
    }
    if ((int32_t)hi < 0) return false;
    drop(1);
    used += 1;
    value = N;
    return true;
  }
};

// Lookup table for the recursive Elias code: entry i (the next 12 stream bits) holds
// value | length << 8 when those bits start with a complete code of at most 12 bits (every value
// below 64), else 0. Built once per CTA with the definition's decoder.
constexpr uint32_t kLutBits = 12;

__device__ __forceinline__ void fill_elias_lut(uint16_t* lut) {
  for (uint32_t i = threadIdx.x; i < (1u << kLutBits); i += blockDim.x) {
    uint32_t w = i << (32 - kLutBits), N = 1, used = 0;
    bool ok = true;
    for (int it = 0; it < 3 && (w >> 31); ++it) {
      const uint32_t nb = N + 1;
      if (used + nb > kLutBits) { ok = false; break; }
      N = w >> (32 - nb);
      w <<= nb;
      used += nb;
    }
    ok = ok && !(w >> 31) && used + 1 <= kLutBits;
    lut[i] = ok ? (uint16_t)(N | ((used + 1) << 8)) : (uint16_t)0;
  }
}

// One Elias integer from the window: table hit in the common case, group loop otherwise.
__device__ __forceinline__ bool read_int(BitSrc& src, const uint16_t* lut, uint32_t skip, uint32_t& value,
                                         uint32_t& used) {
  // `skip` (0 or 1) bits in front of the code are dropped together with it
  const uint32_t e = lut[(src.hi << skip) >> (32 - kLutBits)];
  if (e) {
    const uint32_t nb = (e >> 8) + skip;
    value = e & 0xFFu;
    src.drop(nb);
    used += nb;
    return true;
  }
  if (skip) { src.drop(1); used += 1; }
  return src.elias(value, used);
}

template <int LB, bool DENSE>
__device__ __forceinline__ uint32_t parse_to_fields(const uint32_t* __restrict__ words,
                                                    const uint64_t* __restrict__ table, uint64_t b,
                                                    uint64_t B, uint32_t db, uint32_t d, uint32_t s,
                                                    const uint16_t* lut, uint32_t* __restrict__ row,
                                                    float* A_out) {
  const uint64_t lo = __ldg(table + b), hi = __ldg(table + b + 1), all = __ldg(table + B);
  *A_out = 0.f;
  if (hi < lo || hi - lo < 32 || hi > all) return QSGD_DEV_TABLE;
  const uint64_t cap_bits = (uint64_t)((const uint8_t*)table - (const uint8_t*)words) * 8ull;
  if ((const uint8_t*)table > (const uint8_t*)words && all > cap_bits) return QSGD_DEV_TABLE;
  if (hi - lo > 32ull + (uint64_t)db * 40ull) return QSGD_DEV_OVERRUN;   // longer than any legal string
  const uint32_t total = (uint32_t)(hi - lo) - 32u;
  BitSrc src;
  src.open(words, lo);
  *A_out = __uint_as_float(src.take(32));
  uint32_t* srow = row + ((d * LB) >> 5);            // sign bitmap of this peer row
  uint32_t used = 0, err = 0;
  // The row is zero and only this lane writes it, so fields are OR-ed in place.
  if (DENSE) {
    for (uint32_t c = 0; c < db; ++c) {
      src.refill();
      const uint32_t neg = src.hi >> 31;
      uint32_t v;
      if (!read_int(src, lut, 1u, v, used)) { err = QSGD_DEV_OVERRUN; break; }
      if (used > total) { err = QSGD_DEV_OVERRUN; break; }
      if (v - 1u > s) { err = QSGD_DEV_LEVEL; break; }
      if (v > 1u) {
        row[(c * LB) >> 5] |= (v - 1u) << ((c * LB) & 31);
        if (neg) srow[c >> 5] |= 1u << (c & 31);
      }
    }
    if (!err && used != total) err = QSGD_DEV_OVERRUN;
  } else {
    uint32_t at = 0xFFFFFFFFu;                        // position of the previous nonzero (-1)
    while (used < total && err == 0u) {
      // One refill leaves >= 33 bits: enough for a table-decoded triple (<= 12 + 1 + 12 bits).
      src.refill();
      uint32_t gap, level, neg;
      const uint32_t e1 = lut[src.hi >> (32 - kLutBits)];
      if (e1) {
        gap = e1 & 0xFFu;
        src.drop(e1 >> 8);
        used += e1 >> 8;
      } else {
        if (!src.elias(gap, used)) { err = QSGD_DEV_OVERRUN; break; }
        src.refill();
      }
      neg = src.hi >> 31;
      const uint32_t e2 = lut[(src.hi << 1) >> (32 - kLutBits)];
      if (e2) {
        level = e2 & 0xFFu;
        src.drop((e2 >> 8) + 1u);
        used += (e2 >> 8) + 1u;
      } else {
        src.drop(1);
        used += 1;
        if (!src.elias(level, used)) { err = QSGD_DEV_OVERRUN; break; }
      }
      at += gap;
      err |= at >= db ? QSGD_DEV_POSITION : 0u;
      err |= (level < 1u || level > s) ? QSGD_DEV_LEVEL : 0u;
      err |= used > total ? QSGD_DEV_OVERRUN : 0u;
      if (err == 0u) {
        row[(at * LB) >> 5] |= level << ((at * LB) & 31);
        srow[at >> 5] |= neg << (at & 31);
      }
    }
  }
  return err;
}

template <int LB, bool DENSE, bool FUSED, bool SINGLE>
__global__ void __launch_bounds__(128) decode_elias_fields_kernel(const __grid_constant__ FieldParams p) {
  extern __shared__ __align__(16) uint32_t fsm[];
  __shared__ __align__(16) float xi_tab[LB == 8 ? 256 * 32 : 32];
  __shared__ uint16_t elias_lut[1u << kLutBits];
  const uint32_t tid = threadIdx.x, lane = tid & 31, warp = tid >> 5, nwarps = blockDim.x >> 5;
  const float sf = (float)p.s;
  float lut0 = 0.f;
  fill_elias_lut(elias_lut);
  if (LB == 8) {
    for (uint32_t i = tid; i < 256 * 32; i += blockDim.x) xi_tab[i] = __fdiv_rn((float)(i >> 5), sf);
  }
  __syncthreads();
  if (LB != 8) {
    const uint32_t level = lane & ((1u << LB) - 1u), neg = (lane >> LB) & 1u;
    const float q = __fdiv_rn((float)level, sf);
    lut0 = neg ? -q : q;
  }
  const uint8_t* tab_lane = reinterpret_cast<const uint8_t*>(xi_tab) + 4 * lane;

  const uint32_t warp_words = p.G * p.bucket_words;
  uint32_t* mine = fsm + (size_t)warp * warp_words;
  const uint32_t level_words = (p.d * LB) >> 5;
  const uint32_t pg = lane / p.Kpad, pk = lane % p.Kpad;      // parse role: bucket in group, peer
  const uint32_t slots_per_bucket = p.d >> 4;                 // 16-coordinate lane slots
  const uint32_t total_slots = p.G * slots_per_bucket;
  const uint64_t groups = (p.B + p.G - 1) / p.G;

  for (uint64_t grp = (uint64_t)blockIdx.x * nwarps + warp; grp < groups; grp += (uint64_t)gridDim.x * nwarps) {
    const uint64_t b0 = grp * p.G;
    for (uint32_t q = lane; q < (warp_words >> 2); q += 32) reinterpret_cast<uint4*>(mine)[q] = make_uint4(0u, 0u, 0u, 0u);
    __syncwarp();
    // ---- phase 1: one lane per (bucket, peer) ------------------------------------------------
    for (uint32_t k = pk; k < p.K; k += 32) {
      const uint64_t b = b0 + pg;
      if (pg < p.G && b < p.B) {
        uint32_t* bucket = mine + pg * p.bucket_words;
        const uint64_t base = b * p.d;
        const uint32_t db = (uint32_t)min((uint64_t)p.d, p.n - base);
        float A;
        const uint32_t st = parse_to_fields<LB, DENSE>(p.peers.payload[k], p.peers.table[k], b, p.B, db, p.d,
                                                       p.s, elias_lut, bucket + k * p.row_words, &A);
        reinterpret_cast<float*>(bucket + p.K * p.row_words)[k] = A;
        if (st) atomicOr(p.status, st);
      }
      if (p.Kpad < 32) break;
    }
    __syncwarp();
    // ---- phase 2: the fixed-width decoder's inner loop over the rebuilt fields ----------------
    for (uint32_t s0 = 0; s0 < total_slots; s0 += 32) {
      const uint32_t slot = s0 + lane;
      const uint32_t g = slot / slots_per_bucket, c = (slot - g * slots_per_bucket) << 4;
      const uint64_t b = b0 + g;
      const uint64_t i0 = b * p.d + c;
      const bool live = slot < total_slots && b < p.B && i0 < p.n;
      const uint32_t* bucket = mine + (live ? g : 0) * p.bucket_words;
      const float* scales = reinterpret_cast<const float*>(bucket + p.K * p.row_words);
      float acc[16];
#pragma unroll
      for (int e = 0; e < 16; ++e) acc[e] = 0.f;
#pragma unroll 2
      for (uint32_t k = 0; k < p.K; ++k) {
        const uint32_t* row = bucket + k * p.row_words;
        uint32_t w[4] = {0u, 0u, 0u, 0u};
        uint32_t sb = 0;
        float A = 0.f;
        if (live) {
          A = scales[k];
          sb = (row[level_words + (c >> 5)] >> (c & 31)) & 0xFFFFu;
          if (LB == 8) {
            const uint4 t = *reinterpret_cast<const uint4*>(row + (c >> 2));
            w[0] = t.x; w[1] = t.y; w[2] = t.z; w[3] = t.w;
          } else if (LB == 4) {
            const uint2 t = *reinterpret_cast<const uint2*>(row + (c >> 3));
            w[0] = t.x; w[1] = t.y;
          } else if (LB == 2) {
            w[0] = row[c >> 4];
          } else {
            w[0] = (row[c >> 5] >> (c & 31)) & 0xFFFFu;
          }
        }
        if (LB == 8) add_peer_tab(acc, w, sb, tab_lane, A);
        else if (SINGLE) add_peer_lut<LB, true>(acc, w, sb, __fmul_rn(__shfl_sync(0xffffffffu, A, 0), lut0), A);
        else add_peer_lut<LB, false>(acc, w, sb, lut0, A);
      }
      if (live) store_lane16<FUSED>(p.out + i0, acc, i0, p.n, p.c);
    }
    __syncwarp();
  }
}

template <int LB, bool DENSE>
int launch_fields(FieldParams& p, bool fused, cudaStream_t stream, bool* handled) {
  *handled = false;
  int dev = 0, max_smem = 0, sms = 0;
  cudaGetDevice(&dev);
  cudaDeviceGetAttribute(&max_smem, cudaDevAttrMaxSharedMemoryPerBlockOptin, dev);
  cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev);
  const uint32_t level_words = (p.d * LB) >> 5, sign_words = p.d >> 5;
  p.row_words = (level_words + sign_words + 3u) & ~3u;
  p.bucket_words = (p.K * p.row_words + p.K + 3u) & ~3u;
  uint32_t kpad = 1;
  while (kpad < p.K && kpad < 32) kpad <<= 1;
  p.Kpad = kpad;
  uint32_t G = p.K <= 32 ? 32 / kpad : 1;
  while (G > 1 && (size_t)G * p.bucket_words * 4 > (16u << 10)) G >>= 1;
  p.G = G;
  const size_t per_warp = (size_t)G * p.bucket_words * 4;
  const size_t budget = (size_t)max_smem - (LB == 8 ? 32768 : 128) - 8192 - 1024;
  int warps = 4;
  while (warps > 1 && (size_t)warps * per_warp > (warps == 4 ? (96u << 10) : budget)) warps >>= 1;
  if ((size_t)warps * per_warp > budget) return 0;               // caller falls back to the slow kernel
  const bool single = p.d >= 512 && (p.d & (p.d - 1)) == 0 && LB != 8;
  void (*kern)(FieldParams);
  if (fused) kern = single ? decode_elias_fields_kernel<LB, DENSE, true, true> : decode_elias_fields_kernel<LB, DENSE, true, false>;
  else kern = single ? decode_elias_fields_kernel<LB, DENSE, false, true> : decode_elias_fields_kernel<LB, DENSE, false, false>;
  const size_t smem = (size_t)warps * per_warp;
  cudaError_t e = cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
  if (e != cudaSuccess) return (int)e;
  int occ = 0;
  e = cudaOccupancyMaxActiveBlocksPerMultiprocessor(&occ, kern, warps * 32, smem);
  if (e != cudaSuccess) return (int)e;
  if (occ < 1) occ = 1;
  const uint64_t groups = (p.B + G - 1) / G;
  const uint64_t want = (groups + warps - 1) / warps;
  const uint64_t cap = (uint64_t)sms * occ;
  const uint32_t grid = (uint32_t)(want < cap ? want : cap);
  {
    ScopedKernel sk(kKernDecodeElias, stream);
    kern<<<grid, warps * 32, smem, stream>>>(p);
  }
  *handled = true;
  return (int)cudaGetLastError();
}

template <int LB>
int launch_fields_lb(FieldParams& p, bool dense, bool fused, cudaStream_t stream, bool* handled) {
  return dense ? launch_fields<LB, true>(p, fused, stream, handled) : launch_fields<LB, false>(p, fused, stream, handled);
}

}  // namespace

int launch_decode_elias(const PeerSet& peers, uint32_t K, uint64_t n, uint32_t d, uint32_t s,
                        bool dense, float* acc_or_x, bool fused, float eta, uint32_t* status_dev,
                        cudaStream_t stream) {
  {
    FieldParams f;
    f.peers = peers; f.K = K; f.n = n; f.d = d; f.s = s;
    f.B = (n + d - 1) / d;
    f.out = acc_or_x; f.c = eta / (float)K; f.status = status_dev;
    bool handled = false;
    int st;
    switch (level_bits_for(s)) {
      case 1: st = launch_fields_lb<1>(f, dense, fused, stream, &handled); break;
      case 2: st = launch_fields_lb<2>(f, dense, fused, stream, &handled); break;
      case 4: st = launch_fields_lb<4>(f, dense, fused, stream, &handled); break;
      default: st = launch_fields_lb<8>(f, dense, fused, stream, &handled); break;
    }
    if (handled || st) return st;
  }
  EliasDecodeParams p;
  p.peers = peers; p.K = K; p.Kc = K; p.n = n; p.d = d; p.s = s;
  p.B = (n + d - 1) / d;
  p.out = acc_or_x; p.c = eta / (float)K; p.status = status_dev; p.warp_bytes = 0;
  if (s <= 127) return dense ? launch_slow<uint8_t, true>(p, fused, stream) : launch_slow<uint8_t, false>(p, fused, stream);
  return dense ? launch_slow<uint16_t, true>(p, fused, stream) : launch_slow<uint16_t, false>(p, fused, stream);
}

}  // namespace qsgd
