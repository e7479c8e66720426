// Internals shared by the Elias decoders (elias_decode*.cu): kernel parameter blocks, the regime
// predicate, the bit window over a payload, Elias integer decoding, and the incremental parse of
// one string. The launchers at the end are what elias_decode.cu dispatches to.
#pragma once

#include "decode_common.cuh"
#include "elias_common.cuh"

namespace qsgd {

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

// Work split of the sparse-regime decoder (elias_decode_sparse.cu): a warp owns G <= 32 / Kpad
// buckets and walks each in ranges of R positions; a (bucket, peer) list holds the C entries of one
// range. Fewer buckets per warp (some lanes idle) spread a small problem over more warps: the parse
// is a chain of dependent instructions, so resident warps are what hides its latency.
struct SparseShape {
  uint32_t Kpad;      // lanes per bucket: K rounded up to a power of two
  uint32_t G;         // buckets per warp
  uint32_t R;         // positions per range; G * R <= 2048 sums per warp
  uint32_t C;         // entries per list and range: one per 32 positions, at least 16, a multiple of 4
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
  sh.C = (sh.C + 3u) & ~3u;                // keeps every warp's share of shared memory a multiple of 16 bytes
  return sh;
}

// Where peer k's offset table is and how many payload bits may be read. Ordinary form: the caller
// gave the table pointer; the payload is bounded by the byte count the caller gave, else by the
// table's own address when it sits behind the payload (as Encode writes it), else not at all.
// Packed form: the table sits at byte info[1] of the message, which also is the padded payload
// length; the place must be 16-byte aligned and the whole table must lie inside the bytes the
// caller declared readable. Returns false (nothing may be read) when the packed place is bad.
struct PeerTable {
  const uint64_t* table;
  uint64_t cap_bits;
};

__device__ __forceinline__ bool peer_table(const PeerSet& ps, uint32_t k, uint64_t B, PeerTable* out) {
  const uint8_t* words = reinterpret_cast<const uint8_t*>(ps.payload[k]);
  if (ps.packed) {
    const uint64_t off = __ldg(ps.table[k] + 1);
    const uint64_t need = 8ull * (B + 1ull);
    out->table = nullptr;
    out->cap_bits = 0;
    if ((off & 15ull) || off > ps.bound[k] || ps.bound[k] - off < need) return false;
    out->table = reinterpret_cast<const uint64_t*>(words + off);
    out->cap_bits = 8ull * off;
    return true;
  }
  const uint8_t* t = reinterpret_cast<const uint8_t*>(ps.table[k]);
  out->table = ps.table[k];
  out->cap_bits = ps.bound[k] ? 8ull * ps.bound[k] : (t > words ? 8ull * (uint64_t)(t - words) : ~0ull);
  return true;
}

// First bit and length of bucket b's string of peer k, after every check that can be made before
// the payload is touched: table entries ascending, at least the 32 bits of the scale, the end
// inside the payload (table's last entry, and that entry inside the bound of peer_table), not
// longer than any legal string of db coordinates. err != 0 means: read nothing.
struct StringRef {
  const uint32_t* words;
  uint64_t lo;        // first bit (the scale)
  uint32_t total;     // bits after the scale
  uint32_t err;
};

__device__ __forceinline__ StringRef string_ref(const PeerSet& ps, uint32_t k, uint64_t b, uint64_t B, uint32_t db) {
  StringRef r;
  r.words = ps.payload[k];
  r.lo = 0; r.total = 0; r.err = 0;
  PeerTable pt;
  if (!peer_table(ps, k, B, &pt)) { r.err = QSGD_DEV_TABLE; return r; }
  const uint64_t lo = __ldg(pt.table + b), hi = __ldg(pt.table + b + 1), all = __ldg(pt.table + B);
  if (hi < lo || hi - lo < 32 || hi > all || all > pt.cap_bits) r.err = QSGD_DEV_TABLE;
  else if (hi - lo > 32ull + (uint64_t)db * 40ull) r.err = QSGD_DEV_OVERRUN;
  else { r.lo = lo; r.total = (uint32_t)(hi - lo) - 32u; }
  return r;
}

// Strings short enough for the entry-list decoder? True when the K payloads average less than a
// quarter of a bit per coordinate beyond the scales: an entry of a sparse bucket costs 11 to 14
// bits, so a list with room for one entry per 32 positions then fills to about 60 % on average and
// rarely overflows. Called by every thread of a CTA (it holds CTA barriers): K threads read the K
// payload lengths side by side and add them up in shared memory, so a kernel that only has to stand
// down costs one round of loads per CTA. Same answer in every kernel that asks.
__device__ __forceinline__ bool sparse_regime(const PeerSet& peers, uint32_t K, uint64_t B, uint32_t d) {
  __shared__ unsigned long long total_bits;
  __shared__ uint32_t bad_place;
  if (threadIdx.x == 0) { total_bits = 0ull; bad_place = 0u; }
  __syncthreads();
  // thread k reads peer k's payload length: the K pairs of dependent loads run side by side
  for (uint32_t k = threadIdx.x; k < K; k += blockDim.x) {
    PeerTable pt;
    if (!peer_table(peers, k, B, &pt)) atomicOr(&bad_place, 1u);     // the field decoders report the bad place
    else atomicAdd(&total_bits, (unsigned long long)__ldg(pt.table + B));
  }
  __syncthreads();
  return K <= 32u && bad_place == 0u && total_bits < (uint64_t)K * B * (32ull + d / 4u);
}

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
  uint32_t range;         // byte-code decoder: positions per range
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

// Launchers of the three decoders. `handled` / `launched` report whether a kernel was started (a
// shape can be outside a decoder's reach); the return value is 0 or a cudaError_t.
int launch_elias_slow(EliasDecodeParams& p, bool dense, bool fused, cudaStream_t stream);
int launch_elias_fields(FieldParams& p, bool dense, bool fused, cudaStream_t stream, bool* handled);
int launch_elias_sparse(const PeerSet& peers, uint32_t K, uint64_t n, uint32_t d, uint32_t s, float* out, bool fused,
                        float c, uint32_t* status, bool check_regime, const BucketMap& map, cudaStream_t stream,
                        bool* launched);

}  // namespace qsgd
