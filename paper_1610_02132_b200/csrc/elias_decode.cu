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
  uint32_t defer_sparse;  // a sparse-regime kernel was launched beside this one
  BucketMap map;       // where the buckets live in `out` (per-tensor policy), or no map
};

// Work split of the sparse-regime decoder (defined further down): a warp owns G <= 32 / Kpad
// buckets and walks each in ranges of R positions; a (bucket, peer) list holds the C entries of one
// range. Fewer buckets per warp (some lanes idle) spread a small problem over more warps: the parse
// is a chain of dependent instructions, so resident warps are what hides its latency.
struct SparseShape {
  uint32_t Kpad;      // lanes per bucket: K rounded up to a power of two
  uint32_t G;         // buckets per warp
  uint32_t R;         // positions per range; G * R <= 2048 sums per warp
  uint32_t C;         // entries per list and range: one per 32 positions, at least 16
};

inline SparseShape sparse_shape(uint32_t K, uint32_t d, uint64_t B, uint32_t sms) {
  SparseShape sh;
  sh.Kpad = 1;
  while (sh.Kpad < K && sh.Kpad < 32u) sh.Kpad <<= 1;
  sh.G = 32u / sh.Kpad;
  while (sh.G > 1u && B / sh.G < (uint64_t)sms * 12u) sh.G >>= 1;
  sh.R = 2048u / sh.G;                     // a power of two, >= 64
  if (sh.R > 1024u) sh.R = 1024u;
  if (d <= sh.R) sh.R = d;                 // whole bucket in one range
  sh.C = sh.R / 32u > 16u ? sh.R / 32u : 16u;
  return sh;
}

// Strings short enough for the entry-list decoder? True when the K payloads average less than a
// quarter of a bit per coordinate beyond the scales: an entry of a sparse bucket costs 11 to 14
// bits, so a list with room for one entry per 32 positions then fills to about 60 % on average and
// rarely overflows. Same answer in every thread of every kernel that asks.
__device__ __forceinline__ bool sparse_regime(const PeerSet& peers, uint32_t K, uint64_t B, uint32_t d) {
  if (K > 32u) return false;
  uint64_t bits = 0;
  for (uint32_t k = 0; k < K; ++k) bits += __ldg(peers.table[k] + B);
  return bits < (uint64_t)K * B * (32ull + d / 4u);
}

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
  if (!DENSE && p.defer_sparse && sparse_regime(p.peers, p.K, p.B, p.d)) return;
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
    float* orow = p.out + base;
    uint32_t dbv = db;                                  // coordinates of the bucket that exist in `out`
    bool vec = true;
    if (p.map.src) {
      orow = p.out + __ldg(p.map.src + b);
      dbv = min(db, __ldg(p.map.len + b));
      vec = p.map.quads != 0u;
    }
    for (uint32_t c = lane * 4; c < dbv; c += 128) {
      const float4 a = *reinterpret_cast<const float4*>(acc + c);
      float* o = orow + c;
      if (vec && c + 4 <= dbv) {
        float4 r = a;
        if (FUSED) {
          const float4 x = *reinterpret_cast<const float4*>(o);
          r.x = __fsub_rn(x.x, __fmul_rn(p.c, a.x)); r.y = __fsub_rn(x.y, __fmul_rn(p.c, a.y));
          r.z = __fsub_rn(x.z, __fmul_rn(p.c, a.z)); r.w = __fsub_rn(x.w, __fmul_rn(p.c, a.w));
        }
        *reinterpret_cast<float4*>(o) = r;
      } else {
        const float t[4] = {a.x, a.y, a.z, a.w};
        for (uint32_t j = 0; j < 4 && c + j < dbv; ++j) o[j] = FUSED ? __fsub_rn(o[j], __fmul_rn(p.c, t[j])) : t[j];
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
  uint32_t defer_sparse;  // a sparse-regime kernel was launched beside this one
  BucketMap map;          // where the buckets live in `out` (per-tensor policy), or no map
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

// ------------------------------------------------------------------------------------------------
// Sparse-regime decoder (Section 3.1, "Sparse Regime": few nonzeros per bucket). When the strings
// are short the work should follow the nonzeros, not the coordinates. A warp owns G buckets; lane
// (bucket, peer) walks that peer's string of that bucket once, range by range: for each range of
// R positions it lists the (position, sign, level) entries that fall into it, the K lists of a
// bucket are then added in ascending k into a tile of R sums by the bucket's lanes (entries of one
// list hit distinct positions), and the tile is written out and re-zeroed. An entry past the range
// waits in a register for its range; a list that overflows is continued by its own lane at its
// turn in the k order, adding straight into the tile. In the fused step, groups of four
// coordinates whose sums are all +0 are left untouched: for c >= 0, x - c * (+0) is x bit for bit.
//
// The regime is decided on the device from the payload lengths (no host synchronisation): this
// kernel and the field-rebuilding kernel are launched back to back, each evaluates the same
// predicate, and exactly one of them does the work.
// ------------------------------------------------------------------------------------------------
struct SparseParams {
  PeerSet peers;
  uint32_t K;
  SparseShape sh;
  uint64_t n;
  uint32_t d;
  uint32_t s;
  uint64_t B;
  float* out;
  float c;
  uint32_t* status;
  uint32_t warp_words;   // shared-memory words per warp: G * R sums, 64 of scales and counts, 32 lists
  uint32_t quad_shift;   // log2(R / 4) when R is a power of two, else 32
  uint32_t check_regime; // 0: the host already knows that this kernel is the one to run
  BucketMap map;         // where the buckets live in `out` (per-tensor policy), or no map
};

// The recursive Elias code (Definition A.1) of one integer below 2^16, decoded without branches
// from the next 32 stream bits (most significant first): "0" is 1; otherwise up to three groups
// follow, each one bit longer than the value of the one before and starting with a 1, closed by a
// 0. Returns false when a fourth group starts.
__device__ __forceinline__ bool elias_from_window(uint32_t w, uint32_t& value, uint32_t& len) {
  const uint32_t c0 = w >> 31;
  const uint32_t n1 = w >> 30;                       // first group: 2 bits
  uint32_t r = w << 2;
  const uint32_t c1 = r >> 31;
  const uint32_t l2 = n1 + 1u;                       // second group: 3 or 4 bits
  const uint32_t n2 = r >> (32u - l2);
  r <<= l2;
  const uint32_t c2 = r >> 31;
  const uint32_t l3 = n2 + 1u;                       // third group: up to 16 bits
  const uint32_t n3 = r >> (32u - l3);
  r <<= l3;
  const uint32_t c3 = r >> 31;
  value = c0 ? (c1 ? (c2 ? n3 : n2) : n1) : 1u;
  len = c0 ? (c1 ? (c2 ? 3u + l2 + l3 : 3u + l2) : 3u) : 1u;
  return !(c0 & c1 & c2 & c3);
}

constexpr uint32_t kNoEntry = 0xFFFFFFFFu;           // entries are position | level << 16 | negative << 31

struct LaneParse {           // one peer's string of one bucket, mid-parse
  BitSrc src;
  uint32_t used, total;      // bits consumed / bits of the string after its scale
  uint32_t at;               // position of the last decoded nonzero (-1 before the first)
  uint32_t err;
  uint32_t pend;             // decoded entry that has not been delivered yet, or kNoEntry
};

// Delivers, in order, the entries with position < rend, at most `limit` of them; sink(index within
// this call, entry). Stops early at the end of the string or at an error. Every decode consumes at
// least three bits of a string whose length is known, so the loop is bounded.
template <typename F>
__device__ __forceinline__ uint32_t advance(LaneParse& st, uint32_t rend, uint32_t limit, uint32_t db, uint32_t s,
                                            F&& sink) {
  uint32_t n = 0;
  if (st.pend != kNoEntry) {                          // the entry that an earlier call had to hold back
    if ((st.pend & 0xFFFFu) >= rend || limit == 0u) return 0u;
    sink(0u, st.pend);
    n = 1;
    st.pend = kNoEntry;
  }
  while (st.used < st.total && st.err == 0u) {
    uint32_t gap, level, len;
    st.src.refill();                                  // >= 33 valid bits: a code takes at most 23
    bool ok = elias_from_window(st.src.hi, gap, len);
    st.src.drop(len);
    st.used += len;
    st.src.refill();
    const uint32_t neg = st.src.hi >> 31;
    if ((st.src.hi & 0x40000000u) == 0u) {            // level 1, by far the most frequent in this regime
      level = 1u;
      len = 1u;
    } else {
      ok &= elias_from_window(st.src.hi << 1, level, len);
    }
    st.src.drop(len + 1u);
    st.used += len + 1u;
    st.at += gap;
    if (!ok || st.at >= db || level > s || st.used > st.total) {
      st.err |= ok ? 0u : QSGD_DEV_OVERRUN;
      st.err |= st.at >= db ? QSGD_DEV_POSITION : 0u;
      st.err |= level > s ? QSGD_DEV_LEVEL : 0u;
      st.err |= st.used > st.total ? QSGD_DEV_OVERRUN : 0u;
      break;
    }
    const uint32_t en = st.at | (level << 16) | (neg << 31);
    if (st.at >= rend || n >= limit) {                // past the range, or no room: keep it for the next call
      st.pend = en;
      break;
    }
    sink(n, en);
    ++n;
  }
  return n;
}

template <bool FUSED>
__global__ void __launch_bounds__(256, 2) decode_elias_sparse_kernel(const __grid_constant__ SparseParams p) {
  extern __shared__ __align__(16) uint32_t ssm[];
  __shared__ float xi[256];
  if (p.check_regime && !sparse_regime(p.peers, p.K, p.B, p.d)) return;
  const uint32_t tid = threadIdx.x, lane = tid & 31, warp = tid >> 5, nwarps = blockDim.x >> 5;
  const uint32_t G = p.sh.G, Kpad = p.sh.Kpad, R = p.sh.R, C = p.sh.C;
  for (uint32_t i = tid; i < 256; i += blockDim.x) xi[i] = __fdiv_rn((float)i, (float)p.s);
  // per warp: G tiles of R sums | 32 scales | 32 counts | 32 lists of C entries
  uint32_t* mine = ssm + (size_t)warp * p.warp_words;
  float* tile = reinterpret_cast<float*>(mine);
  float4* tile4 = reinterpret_cast<float4*>(mine);
  float* scales = reinterpret_cast<float*>(mine + G * R);
  uint32_t* counts = mine + G * R + 32;
  uint32_t* lists = mine + G * R + 64;
  for (uint32_t q = lane; q < ((G * R) >> 2); q += 32) tile4[q] = make_float4(0.f, 0.f, 0.f, 0.f);
  __syncthreads();

  const uint32_t pg = lane / Kpad, pk = lane % Kpad;           // this lane's bucket in the group (idle if >= G) and peer
  float* sums = tile + pg * R;                                 // its bucket's tile
  uint32_t* list = lists + lane * C;
  const bool skip_zero = FUSED && p.c >= 0.f;                  // x - c * (+0) == x
  const uint64_t groups = (p.B + G - 1) / G;
  const uint32_t tile_quads = R >> 2;
  constexpr uint32_t kMore = 0x80000000u;
  constexpr int kU = 8;                                        // quads per lane in flight when writing out

  for (uint64_t grp = (uint64_t)blockIdx.x * nwarps + warp; grp < groups; grp += (uint64_t)gridDim.x * nwarps) {
    const uint64_t b0 = grp * G;
    // ---- open this lane's string ---------------------------------------------------------------
    LaneParse st;
    st.used = st.total = st.err = 0u;
    st.at = 0xFFFFFFFFu;
    st.pend = kNoEntry;
    uint32_t db = 0;                                           // coordinates of this lane's bucket
    float A = 0.f;
    float* xrow = p.out + (b0 + pg) * (uint64_t)p.d;            // this lane's bucket in the output
    if (pg < G && b0 + pg < p.B) {
      db = (uint32_t)min((uint64_t)p.d, p.n - (b0 + pg) * p.d);
      if (p.map.src) {                                           // per-tensor policy: the bucket lives elsewhere
        db = min(db, __ldg(p.map.len + b0 + pg));
        xrow = p.out + __ldg(p.map.src + b0 + pg);
      }
    }
    const bool parsing = db != 0u && pk < p.K;
    if (parsing) {
      const uint64_t b = b0 + pg;
      const uint32_t* words = p.peers.payload[pk];
      const uint64_t* table = p.peers.table[pk];
      const uint64_t lo = __ldg(table + b), hi = __ldg(table + b + 1), all = __ldg(table + p.B);
      const uint64_t cap_bits = (uint64_t)((const uint8_t*)table - (const uint8_t*)words) * 8ull;
      if (hi < lo || hi - lo < 32 || hi > all) st.err = QSGD_DEV_TABLE;
      else if ((const uint8_t*)table > (const uint8_t*)words && all > cap_bits) st.err = QSGD_DEV_TABLE;
      else if (hi - lo > 32ull + (uint64_t)db * 40ull) st.err = QSGD_DEV_OVERRUN;   // longer than any legal string
      else {
        st.total = (uint32_t)(hi - lo) - 32u;
        st.src.open(words, lo);
        A = __uint_as_float(st.src.take(32));
      }
    }
    scales[lane] = A;
    const bool bad_scale = !(fabsf(A) <= 3.402823466e+38f);

    for (uint32_t rbeg = 0; rbeg < p.d; rbeg += R) {
      const uint32_t rend = min(rbeg + R, p.d);
      // ---- phase 1: list the entries of this range -------------------------------------------
      uint32_t mycnt = 0;
      if (parsing) {
        mycnt = advance(st, rend, C, db, p.s, [&](uint32_t e, uint32_t en) { list[e] = en; });
        if (st.pend != kNoEntry && (st.pend & 0xFFFFu) < rend) mycnt |= kMore;
      }
      counts[lane] = mycnt;
      // Rare cases that need the careful paths below: a list that overflowed, a non-finite scale.
      const bool odd_range = __any_sync(0xffffffffu, (mycnt & kMore) != 0u || bad_scale);
      __syncwarp();
      // ---- phase 2: each bucket's lanes add its lists in ascending k -------------------------
      for (uint32_t k = 0; k < p.K; ++k) {
        const uint32_t owner = pg * Kpad + k;
        const float Ak = scales[owner];
        const uint32_t cnt = counts[owner];
        if (odd_range) {
          if (!(fabsf(Ak) <= 3.402823466e+38f)) {            // inf or NaN scale: A * 0 is NaN everywhere
            const float z = __fmul_rn(Ak, 0.f);
            for (uint32_t i = rbeg + pk; i < min(rend, db); i += Kpad) sums[i - rbeg] = __fadd_rn(sums[i - rbeg], z);
          }
          __syncwarp();
        }
        const uint32_t* lk = lists + owner * C;
        for (uint32_t e = pk; e < (cnt & ~kMore); e += Kpad) {
          const uint32_t en = lk[e];
          const float v = __fmul_rn(Ak, xi[(en >> 16) & 0xFFu]);
          float* cell = sums + ((en & 0xFFFFu) - rbeg);
          *cell = __fadd_rn(*cell, (int32_t)en < 0 ? -v : v);
        }
        __syncwarp();
        if (odd_range) {                                     // rest of a long list, by its own lane
          if (lane == owner && (cnt & kMore)) {
            advance(st, rend, 0xFFFFFFFFu, db, p.s, [&](uint32_t, uint32_t en) {
              const float v = __fmul_rn(A, xi[(en >> 16) & 0xFFu]);
              float* cell = sums + ((en & 0xFFFFu) - rbeg);
              *cell = __fadd_rn(*cell, (int32_t)en < 0 ? -v : v);
            });
          }
          __syncwarp();
        }
      }
      // ---- phase 3: write the sums out and re-zero the tiles ------------------------------------
      if (skip_zero && !odd_range) {
        // Fused step, c >= 0: only listed positions can hold a nonzero sum. Each lane walks its own
        // list and claims a cell by exchanging it with +0: whoever receives the nonzero sum applies
        // it to x, so a position listed by several peers is updated once. Eight in flight per lane.
        const uint32_t cnt = mycnt;
        for (uint32_t e0 = 0; e0 < cnt; e0 += kU) {
          float v[kU], x[kU];
          uint32_t pos[kU];
#pragma unroll
          for (int u = 0; u < kU; ++u) {
            v[u] = 0.f;
            pos[u] = 0;
            if (e0 + u < cnt) {
              pos[u] = list[e0 + u] & 0xFFFFu;
              v[u] = atomicExch(sums + (pos[u] - rbeg), 0.f);
            }
          }
#pragma unroll
          for (int u = 0; u < kU; ++u)
            if (__float_as_uint(v[u]) != 0u) x[u] = xrow[pos[u]];
#pragma unroll
          for (int u = 0; u < kU; ++u)
            if (__float_as_uint(v[u]) != 0u) xrow[pos[u]] = __fsub_rn(x[u], __fmul_rn(p.c, v[u]));
        }
        __syncwarp();
        continue;
      }
      // Otherwise scan the G ranges (each contiguous in memory). The place and the length of
      // bucket g are held by the lanes that parse it.
      const uint32_t range_quads = (rend - rbeg) >> 2;
      const bool vec_ok = !p.map.src || p.map.quads != 0u;
      const uint64_t my_row = (uint64_t)(xrow - p.out);
      for (uint32_t q0 = 0; q0 < G * tile_quads; q0 += 32 * kU) {
        float4 t[kU], x[kU];
        uint64_t at[kU];
        uint32_t cnt[kU];                                   // values of the quad to write (0: none)
        uint32_t full = 0;
#pragma unroll
        for (int u = 0; u < kU; ++u) {
          const uint32_t q = q0 + u * 32 + lane;
          const uint32_t g = p.quad_shift < 32u ? q >> p.quad_shift : q / tile_quads;
          const uint32_t j = q - g * tile_quads;
          const uint64_t row = __shfl_sync(0xffffffffu, my_row, (int)(g * Kpad));
          const uint32_t dbg = __shfl_sync(0xffffffffu, db, (int)(g * Kpad));
          const uint32_t pos = rbeg + 4u * j;
          at[u] = row + pos;
          cnt[u] = 0;
          t[u] = make_float4(0.f, 0.f, 0.f, 0.f);
          if (q < G * tile_quads && j < range_quads && pos < dbg) {
            t[u] = tile4[q];
            const bool any = ((__float_as_uint(t[u].x) | __float_as_uint(t[u].y) | __float_as_uint(t[u].z) | __float_as_uint(t[u].w)) != 0u);
            if (any) tile4[q] = make_float4(0.f, 0.f, 0.f, 0.f);
            if (any || !skip_zero) {
              cnt[u] = min(4u, dbg - pos);
              if (cnt[u] == 4u && vec_ok) full |= 1u << u;
            }
          }
        }
        if (FUSED) {
#pragma unroll
          for (int u = 0; u < kU; ++u)
            if ((full >> u) & 1u) x[u] = *reinterpret_cast<const float4*>(p.out + at[u]);
        }
#pragma unroll
        for (int u = 0; u < kU; ++u) {
          if (cnt[u] == 0u) continue;
          float* o = p.out + at[u];
          if ((full >> u) & 1u) {
            float4 r = t[u];
            if (FUSED) {
              r.x = __fsub_rn(x[u].x, __fmul_rn(p.c, r.x)); r.y = __fsub_rn(x[u].y, __fmul_rn(p.c, r.y));
              r.z = __fsub_rn(x[u].z, __fmul_rn(p.c, r.z)); r.w = __fsub_rn(x[u].w, __fmul_rn(p.c, r.w));
            }
            *reinterpret_cast<float4*>(o) = r;
          } else {                                            // a ragged end, or a place that is not 16-byte aligned
            o[0] = FUSED ? __fsub_rn(o[0], __fmul_rn(p.c, t[u].x)) : t[u].x;
            if (cnt[u] > 1u) o[1] = FUSED ? __fsub_rn(o[1], __fmul_rn(p.c, t[u].y)) : t[u].y;
            if (cnt[u] > 2u) o[2] = FUSED ? __fsub_rn(o[2], __fmul_rn(p.c, t[u].z)) : t[u].z;
            if (cnt[u] > 3u) o[3] = FUSED ? __fsub_rn(o[3], __fmul_rn(p.c, t[u].w)) : t[u].w;
          }
        }
      }
      __syncwarp();
    }
    // a string must end exactly where the table says
    if (parsing && st.err == 0u && (st.used != st.total || st.pend != kNoEntry)) st.err = QSGD_DEV_OVERRUN;
    if (st.err) atomicOr(p.status, st.err);
    __syncwarp();
  }
}

// Launches the sparse-regime kernel when the configuration allows one (K <= 32, Code_s); the
// caller then tells the other decoders to stand down when the predicate holds.
int launch_sparse(const PeerSet& peers, uint32_t K, uint64_t n, uint32_t d, uint32_t s, float* out, bool fused,
                  float c, uint32_t* status, bool check_regime, const BucketMap& map, cudaStream_t stream,
                  bool* launched) {
  *launched = false;
  if (K > 32u) return 0;
  int dev = 0, sms = 0;
  cudaGetDevice(&dev);
  cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev);
  SparseParams p;
  p.peers = peers; p.K = K; p.n = n; p.d = d; p.s = s;
  p.B = (n + d - 1) / d;
  p.sh = sparse_shape(K, d, p.B, (uint32_t)sms);
  p.out = out; p.c = c; p.status = status; p.check_regime = check_regime ? 1u : 0u; p.map = map;
  p.warp_words = p.sh.G * p.sh.R + 64u + p.sh.G * p.sh.Kpad * p.sh.C;
  p.quad_shift = 32;
  const uint32_t tile_quads = p.sh.R >> 2;
  if ((tile_quads & (tile_quads - 1)) == 0)
    for (p.quad_shift = 0; (1u << p.quad_shift) < tile_quads; ++p.quad_shift) {}
  const size_t per_warp = (size_t)p.warp_words * 4;              // at most 16.3 KB
  // Warps per CTA: on a problem of about one wave, the count that spreads the warps most evenly
  // over the SMs (the busiest SM sets the time); 8, or 4 when 8 do not fit, otherwise.
  const uint64_t all_groups = (p.B + p.sh.G - 1) / p.sh.G;
  int warps = 8 * per_warp <= (100u << 10) ? 8 : 4;
  if (all_groups <= (uint64_t)sms * 32u) {
    uint64_t best = ~0ull;
    for (int w = warps; w >= 4; --w) {
      const uint64_t ctas = (all_groups + w - 1) / w;
      const uint64_t busiest = (ctas + sms - 1) / sms * w;      // warps on the fullest SM
      if (busiest < best) { best = busiest; warps = w; }
    }
  }
  auto kern = fused ? decode_elias_sparse_kernel<true> : decode_elias_sparse_kernel<false>;
  const size_t smem = (size_t)warps * per_warp;
  cudaError_t e = cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
  if (e != cudaSuccess) return (int)e;
  int occ = 0;
  e = cudaOccupancyMaxActiveBlocksPerMultiprocessor(&occ, kern, warps * 32, smem);
  if (e != cudaSuccess) return (int)e;
  if (occ < 1) occ = 1;
  const uint64_t groups = (p.B + p.sh.G - 1) / p.sh.G;
  const uint64_t want = (groups + warps - 1) / warps;
  const uint64_t cap = (uint64_t)sms * occ;
  const uint32_t grid = (uint32_t)(want < cap ? want : cap);
  {
    ScopedKernel sk(kKernDecodeEliasSparse, stream);
    kern<<<grid, warps * 32, smem, stream>>>(p);
  }
  *launched = true;
  return (int)cudaGetLastError();
}

template <int LB, bool DENSE, bool FUSED, bool SINGLE>
__global__ void __launch_bounds__(320) decode_elias_fields_kernel(const __grid_constant__ FieldParams p) {
  extern __shared__ __align__(16) uint32_t fsm[];
  __shared__ __align__(16) float xi_tab[LB == 8 ? 256 * 32 : 32];
  __shared__ uint16_t elias_lut[1u << kLutBits];
  if (!DENSE && p.defer_sparse && sparse_regime(p.peers, p.K, p.B, p.d)) return;
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
      if (live) {
        if (p.map.src) store_span16<FUSED>(out_span(p.out, p.map, b, c, p.d, p.n, 16u), acc, p.c);
        else store_lane16<FUSED>(p.out + i0, acc, i0, p.n, p.c);
      }
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
  // Warps per CTA: the count that leaves the most warps resident on an SM. The code table and the
  // level table are per CTA, the fields per warp; the parse is latency-bound, so warps are what counts.
  const size_t per_cta = (LB == 8 ? 32768 : 128) + 8192 + 1024;
  const size_t per_sm = 227u << 10;
  int warps = 0, best = 0;
  for (int w = 1; w <= 10; ++w) {
    if ((size_t)w * per_warp > budget) break;
    const int resident = (int)(per_sm / ((size_t)w * per_warp + per_cta)) * w;
    if (resident > best) { best = resident; warps = w; }
  }
  if (warps == 0) return 0;                                      // caller falls back to the slow kernel
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

// ------------------------------------------------------------------------------------------------
// Field-rebuilding decoder for long buckets (d >= 1024): the same two phases, but a bucket is
// walked in ranges of 512 positions. A lane keeps its place in its string between ranges (bit
// window, position, one decoded entry that lies past the range), so shared memory holds the fields
// of one range only and as many warps fit on an SM as for d = 512; with whole-bucket fields a CTA
// of d = 4096 is down to one or two warps.
// ------------------------------------------------------------------------------------------------
template <int LB, bool DENSE, bool FUSED>
__global__ void __launch_bounds__(128) decode_elias_ranged_kernel(const __grid_constant__ FieldParams p) {
  constexpr uint32_t kR = 512;                                  // positions per range = one warp pass of phase 2
  constexpr uint32_t kLevelWords = kR * LB / 32, kRowWords = kLevelWords + kR / 32;
  extern __shared__ __align__(16) uint32_t fsm[];
  __shared__ __align__(16) float xi_tab[LB == 8 ? 256 * 32 : 32];
  if (!DENSE && p.defer_sparse && sparse_regime(p.peers, p.K, p.B, p.d)) return;
  const uint32_t tid = threadIdx.x, lane = tid & 31, warp = tid >> 5, nwarps = blockDim.x >> 5;
  const float sf = (float)p.s;
  float lut0 = 0.f;
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

  // per warp: G * K rows of kRowWords (level fields, then sign bits, of one range) | 32 scales
  const uint32_t rows_words = p.G * p.K * kRowWords;
  uint32_t* mine = fsm + (size_t)warp * (rows_words + 32u);
  float* scales = reinterpret_cast<float*>(mine + rows_words);
  const uint32_t pg = lane / p.Kpad, pk = lane % p.Kpad;      // parse role: bucket in group, peer
  uint32_t* row = mine + (pg * p.K + pk) * kRowWords;         // this lane's row (when it parses)
  const uint64_t groups = (p.B + p.G - 1) / p.G;

  for (uint64_t grp = (uint64_t)blockIdx.x * nwarps + warp; grp < groups; grp += (uint64_t)gridDim.x * nwarps) {
    const uint64_t b0 = grp * p.G;
    // ---- open this lane's string ---------------------------------------------------------------
    LaneParse st;
    st.used = st.total = st.err = 0u;
    st.at = 0xFFFFFFFFu;
    st.pend = kNoEntry;
    uint32_t db = 0;
    float A = 0.f;
    if (pg < p.G && b0 + pg < p.B) db = (uint32_t)min((uint64_t)p.d, p.n - (b0 + pg) * p.d);
    const bool parsing = db != 0u && pk < p.K;
    if (parsing) {
      const uint64_t b = b0 + pg;
      const uint32_t* words = p.peers.payload[pk];
      const uint64_t* table = p.peers.table[pk];
      const uint64_t lo = __ldg(table + b), hi = __ldg(table + b + 1), all = __ldg(table + p.B);
      const uint64_t cap_bits = (uint64_t)((const uint8_t*)table - (const uint8_t*)words) * 8ull;
      if (hi < lo || hi - lo < 32 || hi > all) st.err = QSGD_DEV_TABLE;
      else if ((const uint8_t*)table > (const uint8_t*)words && all > cap_bits) st.err = QSGD_DEV_TABLE;
      else if (hi - lo > 32ull + (uint64_t)db * 40ull) st.err = QSGD_DEV_OVERRUN;   // longer than any legal string
      else {
        st.total = (uint32_t)(hi - lo) - 32u;
        st.src.open(words, lo);
        A = __uint_as_float(st.src.take(32));
      }
    }
    scales[lane] = A;
    const bool readable = parsing && st.err == 0u;

    for (uint32_t rbeg = 0; rbeg < p.d; rbeg += kR) {
      const uint32_t rend = min(rbeg + kR, p.d);
      for (uint32_t q = lane; q < (rows_words >> 2); q += 32) reinterpret_cast<uint4*>(mine)[q] = make_uint4(0u, 0u, 0u, 0u);
      __syncwarp();
      // ---- phase 1: this lane's entries of the range, OR-ed into its zeroed row ----------------
      if (readable) {
        uint32_t* srow = row + kLevelWords;
        if (DENSE) {
          for (uint32_t c = rbeg; c < min(rend, db) && st.err == 0u; ++c) {
            st.src.refill();
            const uint32_t neg = st.src.hi >> 31;
            uint32_t v, len;
            const bool ok = elias_from_window(st.src.hi << 1, v, len);
            st.src.drop(len + 1u);
            st.used += len + 1u;
            if (!ok || st.used > st.total) st.err = QSGD_DEV_OVERRUN;
            else if (v - 1u > p.s) st.err = QSGD_DEV_LEVEL;
            else if (v > 1u) {
              const uint32_t pos = c - rbeg;
              row[(pos * LB) >> 5] |= (v - 1u) << ((pos * LB) & 31);
              srow[pos >> 5] |= neg << (pos & 31);
            }
          }
        } else {
          advance(st, rend, 0xFFFFFFFFu, db, p.s, [&](uint32_t, uint32_t en) {
            const uint32_t pos = (en & 0xFFFFu) - rbeg;
            row[(pos * LB) >> 5] |= ((en >> 16) & 0xFFu) << ((pos * LB) & 31);
            srow[pos >> 5] |= (en >> 31) << (pos & 31);
          });
        }
      }
      __syncwarp();
      // ---- phase 2: one warp pass per bucket over the range's fields, ascending k ---------------
      for (uint32_t g = 0; g < p.G; ++g) {
        const uint64_t b = b0 + g;
        const uint32_t cl = lane << 4, c = rbeg + cl;           // position in the range / in the bucket
        const uint64_t i0 = b * p.d + c;
        const bool live = b < p.B && c < rend && i0 < p.n;
        if (!__any_sync(0xffffffffu, live)) continue;
        float acc[16];
#pragma unroll
        for (int e = 0; e < 16; ++e) acc[e] = 0.f;
#pragma unroll 2
        for (uint32_t k = 0; k < p.K; ++k) {
          const uint32_t* rk = mine + (g * p.K + k) * kRowWords;
          uint32_t w[4] = {0u, 0u, 0u, 0u};
          uint32_t sb = 0;
          const float Ak = scales[g * p.Kpad + k];
          if (live) {
            sb = (rk[kLevelWords + (cl >> 5)] >> (cl & 31)) & 0xFFFFu;
            if (LB == 8) {
              const uint4 t = *reinterpret_cast<const uint4*>(rk + (cl >> 2));
              w[0] = t.x; w[1] = t.y; w[2] = t.z; w[3] = t.w;
            } else if (LB == 4) {
              const uint2 t = *reinterpret_cast<const uint2*>(rk + (cl >> 3));
              w[0] = t.x; w[1] = t.y;
            } else if (LB == 2) {
              w[0] = rk[cl >> 4];
            } else {
              w[0] = (rk[cl >> 5] >> (cl & 31)) & 0xFFFFu;
            }
          }
          if (LB == 8) add_peer_tab(acc, w, sb, tab_lane, live ? Ak : 0.f);
          else add_peer_lut<LB, true>(acc, w, sb, __fmul_rn(Ak, lut0), Ak);
        }
        if (live) {
          if (p.map.src) store_span16<FUSED>(out_span(p.out, p.map, b, c, p.d, p.n, 16u), acc, p.c);
          else store_lane16<FUSED>(p.out + i0, acc, i0, p.n, p.c);
        }
      }
      __syncwarp();
    }
    // a string must end exactly where the table says
    if (readable && st.err == 0u && (st.used != st.total || st.pend != kNoEntry)) st.err = QSGD_DEV_OVERRUN;
    if (st.err) atomicOr(p.status, st.err);
    __syncwarp();
  }
}

template <int LB, bool DENSE>
int launch_ranged(FieldParams& p, bool fused, cudaStream_t stream, bool* handled) {
  *handled = false;
  if (p.K > 32u) return 0;
  int dev = 0, sms = 0;
  cudaGetDevice(&dev);
  cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev);
  constexpr uint32_t kRowWords = 512u * LB / 32u + 16u;
  uint32_t kpad = 1;
  while (kpad < p.K) kpad <<= 1;
  p.Kpad = kpad;
  p.G = 32u / kpad;
  const size_t per_warp = ((size_t)p.G * p.K * kRowWords + 32u) * 4;   // at most 18.6 KB
  const int warps = 4;
  auto kern = fused ? decode_elias_ranged_kernel<LB, DENSE, true> : decode_elias_ranged_kernel<LB, DENSE, false>;
  const size_t smem = (size_t)warps * per_warp;
  cudaError_t e = cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
  if (e != cudaSuccess) return (int)e;
  int occ = 0;
  e = cudaOccupancyMaxActiveBlocksPerMultiprocessor(&occ, kern, warps * 32, smem);
  if (e != cudaSuccess) return (int)e;
  if (occ < 1) occ = 1;
  const uint64_t groups = (p.B + p.G - 1) / p.G;
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
  if (p.d >= 1024u && p.K <= 32u)       // long buckets: fields of one range at a time
    return dense ? launch_ranged<LB, true>(p, fused, stream, handled) : launch_ranged<LB, false>(p, fused, stream, handled);
  return dense ? launch_fields<LB, true>(p, fused, stream, handled) : launch_fields<LB, false>(p, fused, stream, handled);
}

}  // namespace

int launch_decode_elias(const PeerSet& peers, uint32_t K, uint64_t n, uint32_t d, uint32_t s,
                        bool dense, float* acc_or_x, bool fused, float eta, uint32_t* status_dev,
                        const BucketMap& map, cudaStream_t stream) {
  // Which decoder? In a message the offset table follows the padded payload, so table - payload is
  // the payload size and the host can evaluate the regime predicate itself (to within the padding)
  // and launch one kernel. With tables kept elsewhere the sizes are only known on the device: both
  // kernels are launched and exactly one does the work. Either decoder is correct on any input;
  // the choice is about speed only.
  const uint64_t B = (n + d - 1) / d;
  bool sizes_known = !dense && K <= 32u;
  uint64_t payload_bits = 0;
  for (uint32_t k = 0; k < K && sizes_known; ++k) {
    const uint8_t* w = reinterpret_cast<const uint8_t*>(peers.payload[k]);
    const uint8_t* t = reinterpret_cast<const uint8_t*>(peers.table[k]);
    const uint64_t longest = align16((B * 32ull + n * 40ull + 7ull) / 8ull);   // no legal payload is longer
    if (t <= w || (uint64_t)(t - w) > longest) sizes_known = false;
    else payload_bits += 8ull * (uint64_t)(t - w);
  }
  const bool host_sparse = sizes_known && payload_bits < (uint64_t)K * B * (32ull + d / 4u);
  bool sparse = false;
  {
    FieldParams f;
    f.peers = peers; f.K = K; f.n = n; f.d = d; f.s = s;
    f.B = B;
    f.out = acc_or_x; f.c = eta / (float)K; f.status = status_dev; f.map = map;
    bool handled = false;
    int st = 0;
    if (!dense && (host_sparse || !sizes_known))
      st = launch_sparse(peers, K, n, d, s, acc_or_x, fused, f.c, status_dev, !sizes_known, map, stream, &sparse);
    if (st) return st;
    if (sparse && sizes_known) return 0;                    // the host chose the sparse-regime kernel
    f.defer_sparse = sparse ? 1u : 0u;
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
  p.defer_sparse = sparse ? 1u : 0u; p.map = map;
  if (s <= 127) return dense ? launch_slow<uint8_t, true>(p, fused, stream) : launch_slow<uint8_t, false>(p, fused, stream);
  return dense ? launch_slow<uint16_t, true>(p, fused, stream) : launch_slow<uint16_t, false>(p, fused, stream);
}

}  // namespace qsgd
