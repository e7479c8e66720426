// QSGD oracle: a plain, slow, single-threaded CPU statement of the quantizer Q_s, the
// fixed-width and Elias-coded messages, Decode, the K-peer aggregate and the SGD step.
//
// THIS IS TEST INFRASTRUCTURE, NOT PRODUCT CODE. Only the test-suite, the smoke check and the
// CPU-baseline leg of the benchmark may load it. It shares no code, header, table or constant
// generator with the CUDA path and is written from the paper's text alone.
//
// Build: g++ -std=c++17 -O2 -ffp-contract=off -fno-fast-math -shared -fPIC
// (no FMA contraction, no flush-to-zero: every fp32 operation below is one IEEE-754
// round-to-nearest-even operation, in the order written).
//
// Passages followed (QSGD, arXiv 1610.02132):
//   Section 3.1, Eq. (2)              stochastic quantizer Q_s
//   Section 3.1 "Efficient Coding"    tuple (norm, sigma, zeta), string S (= Code_s)
//   Appendix A.2, Definition A.1      recursive Elias coding, encoder and decoder
//   Appendix A.3                      Code'_s: every coordinate, Elias(level + 1)
//   Section 4 (Experiments)           buckets of d consecutive values, max-norm scaling
//   Algorithm 1                       decode K peers, x <- x - (eta/K) * sum
//
// Pins (tests, CPU only): Lemma 3.1 (unbiasedness, variance, sparsity) by Monte-Carlo and by
// exhaustive enumeration for n <= 8; textbook Elias-omega code words; the paper's encoder and
// decoder checked against each other; lossless round trip; Philox4x32-10 against an independent
// library engine. The fixed-width layout, the per-bucket offset table, the bit order of the
// stream, the canonical sign of a zero level and the ascending-k summation order are format
// choices of this implementation, not of the paper: for those, PARITY IS UNPINNED with respect
// to the paper and pinned only by round trip.

#include <cmath>
#include <cstdint>
#include <cstring>
#include <string>
#include <vector>

namespace {

// ---------------------------------------------------------------------------------------------
// Philox4x32-10 (Salmon, Moraes, Dror, Shaw: "Parallel random numbers: as easy as 1, 2, 3").
// Ten rounds; the key is advanced by the Weyl constants between rounds.
// ---------------------------------------------------------------------------------------------
void philox_round(uint32_t c[4], const uint32_t k[2]) {
  const uint64_t p0 = (uint64_t)0xD2511F53u * (uint64_t)c[0];
  const uint64_t p1 = (uint64_t)0xCD9E8D57u * (uint64_t)c[2];
  const uint32_t n0 = (uint32_t)(p1 >> 32) ^ c[1] ^ k[0];
  const uint32_t n1 = (uint32_t)p1;
  const uint32_t n2 = (uint32_t)(p0 >> 32) ^ c[3] ^ k[1];
  const uint32_t n3 = (uint32_t)p0;
  c[0] = n0; c[1] = n1; c[2] = n2; c[3] = n3;
}

void philox4x32_10(const uint32_t ctr[4], const uint32_t key[2], uint32_t out[4]) {
  uint32_t c[4] = {ctr[0], ctr[1], ctr[2], ctr[3]};
  uint32_t k[2] = {key[0], key[1]};
  for (int r = 0; r < 10; ++r) {
    if (r > 0) { k[0] += 0x9E3779B9u; k[1] += 0xBB67AE85u; }
    philox_round(c, k);
  }
  for (int j = 0; j < 4; ++j) out[j] = c[j];
}

// Uniform in [0, 1 - 2^-24] for the coordinate with GLOBAL index i: block q = i / 4 of the
// stream keyed by (seed) and positioned by (step, worker); word i % 4; top 24 bits.
float uniform01(uint64_t seed, uint32_t step, uint32_t worker, uint64_t i) {
  const uint64_t q = i >> 2;
  const uint32_t ctr[4] = {(uint32_t)q, (uint32_t)(q >> 32), step, worker};
  const uint32_t key[2] = {(uint32_t)seed, (uint32_t)(seed >> 32)};
  uint32_t x[4];
  philox4x32_10(ctr, key, x);
  const uint32_t m = x[i & 3] >> 8;             // 24-bit integer, exact in fp32
  return (float)m * 5.9604644775390625e-08f;    // * 2^-24, exact
}

int level_bits(uint32_t s) {                     // field width of the fixed-width code
  if (s <= 1) return 1;
  if (s <= 3) return 2;
  if (s <= 15) return 4;
  return 8;
}

uint64_t align16(uint64_t x) { return (x + 15u) & ~(uint64_t)15u; }

uint64_t n_buckets(uint64_t n, uint32_t d) { return (n + d - 1) / d; }

// ---------------------------------------------------------------------------------------------
// Bucket scale (Eq. 2: ||v||_2; Section 4: max |v_i|). A scale below the smallest normal fp32
// (zero included) marks a zero bucket: Q(0) = 0.
// ---------------------------------------------------------------------------------------------
float bucket_scale(const float* v, uint64_t len, int norm_kind) {
  float A;
  if (norm_kind == 0) {
    double acc = 0.0;
    for (uint64_t j = 0; j < len; ++j) acc += (double)v[j] * (double)v[j];
    A = (float)std::sqrt(acc);
  } else {
    A = 0.0f;
    for (uint64_t j = 0; j < len; ++j) { const float a = std::fabs(v[j]); if (a > A) A = a; }
  }
  if (!(A >= 1.17549435e-38f)) A = 0.0f;
  return A;
}

// Level and sign of one coordinate given its bucket scale (Eq. 2, with the rounding fixed):
//   t = (s * |v|) * (1 / A);  c = t + u;  level = min(floor(c), s);  sign only if level > 0.
void quantize_one(float v, float A, uint32_t s, float u, uint32_t* level, uint32_t* sign) {
  if (!(A >= 1.17549435e-38f)) { *level = 0; *sign = 0; return; }
  const float sf = (float)s;
  const float r = 1.0f / A;
  const float a = std::fabs(v);
  float t = sf * a;
  t = t * r;
  const float c = t + u;
  uint32_t l = (uint32_t)(int32_t)c;            // c >= 0: truncation is floor
  if (l > s) l = s;
  *level = l;
  *sign = (l > 0 && v < 0.0f) ? 1u : 0u;
}

// Reconstruction (Eq. 2): A * sgn * (level / s); level / s first, then one multiply.
float dequantize_one(float A, uint32_t s, uint32_t level, uint32_t sign) {
  const float xi = (float)level / (float)s;
  const float m = A * xi;
  return sign ? -m : m;
}

// ---------------------------------------------------------------------------------------------
// Bit stream: bit t of the stream is bit (31 - t % 32) of little-endian u32 word t / 32.
// ---------------------------------------------------------------------------------------------
struct BitWriter {
  uint32_t* words; uint64_t cap_bits; uint64_t pos; bool overflow;
  void put(int bit) {
    if (pos >= cap_bits) { overflow = true; ++pos; return; }
    if (bit) words[pos >> 5] |= (uint32_t)1u << (31 - (pos & 31));
    ++pos;
  }
  void put_str(const std::string& s) { for (char ch : s) put(ch == '1'); }
};

struct BitReader {
  const uint32_t* words; uint64_t pos; uint64_t end; bool fail;
  int get() {
    if (pos >= end) { fail = true; return 0; }
    const int b = (int)((words[pos >> 5] >> (31 - (pos & 31))) & 1u);
    ++pos;
    return b;
  }
};

// Definition A.1, encoder. The printed termination test reads "k = 0"; with that test the code
// of 1 would be "10", which the printed decoder reads as 2. The test that makes encoder and
// decoder inverse (and gives |Elias(1)| = 1, the lemma's length) is k = 1.
std::string elias_string(uint64_t k) {
  std::string s = "0";
  while (k > 1) {
    std::string bin;
    for (uint64_t t = k; t > 0; t >>= 1) bin.insert(bin.begin(), (t & 1) ? '1' : '0');
    s = bin + s;
    k = (uint64_t)bin.size() - 1;
  }
  return s;
}

// Definition A.1, decoder: N = 1; while the next bit is 1, that bit and N more bits form the
// new N; a 0 ends the code. Values that need more than 32 bits are rejected.
uint64_t elias_read(BitReader& br) {
  uint64_t N = 1;
  for (;;) {
    const int b = br.get();
    if (br.fail) return 0;
    if (b == 0) return N;
    if (N > 31) { br.fail = true; return 0; }
    uint64_t v = 1;
    for (uint64_t j = 0; j < N; ++j) { v = (v << 1) | (uint64_t)br.get(); if (br.fail) return 0; }
    N = v;
  }
}

uint32_t float_bits(float f) { uint32_t u; std::memcpy(&u, &f, 4); return u; }
float bits_float(uint32_t u) { float f; std::memcpy(&f, &u, 4); return f; }

}  // namespace

extern "C" {

enum { OQ_NORM_L2 = 0, OQ_NORM_MAX = 1 };
enum { OQ_CODE_FIXED = 0, OQ_CODE_ELIAS = 1, OQ_CODE_ELIAS_DENSE = 2 };

void oq_philox4x32_10(const uint32_t* ctr, const uint32_t* key, uint32_t* out) {
  philox4x32_10(ctr, key, out);
}

float oq_uniform(uint64_t seed, uint32_t step, uint32_t worker, uint64_t i) {
  return uniform01(seed, step, worker, i);
}

int oq_level_bits(uint32_t s) { return level_bits(s); }

// Scales of all buckets of g[0..n).
void oq_bucket_scales(const float* g, uint64_t n, uint32_t d, int norm_kind, float* A) {
  const uint64_t B = n_buckets(n, d);
  for (uint64_t b = 0; b < B; ++b) {
    const uint64_t lo = b * d, hi = (lo + d < n) ? lo + d : n;
    A[b] = bucket_scale(g + lo, hi - lo, norm_kind);
  }
}

// Levels and signs of g[0..n) given the bucket scales A (the oracle's own, or scales emitted
// by another implementation). i0 is the global index of g[0] (a multiple of d) so that a slice
// of a large gradient draws the same uniforms as the whole.
void oq_quantize(const float* g, uint64_t n, uint32_t d, uint32_t s, const float* A,
                 uint64_t seed, uint32_t step, uint32_t worker, uint64_t i0,
                 uint8_t* levels, uint8_t* signs) {
  for (uint64_t i = 0; i < n; ++i) {
    const float u = uniform01(seed, step, worker, i0 + i);
    uint32_t l, sg;
    quantize_one(g[i], A[i / d], s, u, &l, &sg);
    levels[i] = (uint8_t)l;
    signs[i] = (uint8_t)sg;
  }
}

// Same, but with the uniforms supplied (for enumeration tests that choose u directly).
void oq_quantize_with_uniforms(const float* g, uint64_t n, uint32_t d, uint32_t s, const float* A,
                               const float* u, uint8_t* levels, uint8_t* signs) {
  for (uint64_t i = 0; i < n; ++i) {
    uint32_t l, sg;
    quantize_one(g[i], A[i / d], s, u[i], &l, &sg);
    levels[i] = (uint8_t)l;
    signs[i] = (uint8_t)sg;
  }
}

// Q_s values from the tuple (A, sigma, zeta).
void oq_dequantize(const float* A, const uint8_t* levels, const uint8_t* signs, uint64_t n,
                   uint32_t d, uint32_t s, float* out) {
  for (uint64_t i = 0; i < n; ++i) out[i] = dequantize_one(A[i / d], s, levels[i], signs[i]);
}

// ------------------------------- fixed-width message ----------------------------------------
// Regions, each zero-padded to a multiple of 16 bytes: A[B] fp32 | sign bitmap | level fields.
// layout[0] = byte offset of the sign bitmap, [1] = byte offset of the level fields,
// [2] = total bytes, [3] = level bits per coordinate.
void oq_fixed_layout(uint64_t n, uint32_t d, uint32_t s, uint64_t* layout) {
  const uint64_t B = n_buckets(n, d);
  const uint64_t lb = (uint64_t)level_bits(s);
  const uint64_t a = align16(4 * B);
  const uint64_t sg = align16(4 * ((n + 31) / 32));
  const uint64_t lv = align16(4 * ((n * lb + 31) / 32));
  layout[0] = a; layout[1] = a + sg; layout[2] = a + sg + lv; layout[3] = lb;
}

void oq_fixed_pack(const float* A, const uint8_t* levels, const uint8_t* signs, uint64_t n,
                   uint32_t d, uint32_t s, uint8_t* out) {
  uint64_t lay[4];
  oq_fixed_layout(n, d, s, lay);
  std::memset(out, 0, lay[2]);
  const uint64_t B = n_buckets(n, d);
  std::memcpy(out, A, 4 * B);
  uint32_t* sw = (uint32_t*)(out + lay[0]);
  uint32_t* lw = (uint32_t*)(out + lay[1]);
  const uint64_t lb = lay[3];
  for (uint64_t i = 0; i < n; ++i) {
    if (signs[i]) sw[i / 32] |= (uint32_t)1u << (i % 32);
    const uint64_t bit = i * lb;
    lw[bit / 32] |= (uint32_t)levels[i] << (bit % 32);
  }
}

void oq_fixed_unpack(const uint8_t* msg, uint64_t n, uint32_t d, uint32_t s, float* A,
                     uint8_t* levels, uint8_t* signs) {
  uint64_t lay[4];
  oq_fixed_layout(n, d, s, lay);
  const uint64_t B = n_buckets(n, d);
  std::memcpy(A, msg, 4 * B);
  const uint32_t* sw = (const uint32_t*)(msg + lay[0]);
  const uint32_t* lw = (const uint32_t*)(msg + lay[1]);
  const uint64_t lb = lay[3];
  const uint32_t mask = (lb == 32) ? 0xFFFFFFFFu : (((uint32_t)1u << lb) - 1u);
  for (uint64_t i = 0; i < n; ++i) {
    signs[i] = (uint8_t)((sw[i / 32] >> (i % 32)) & 1u);
    const uint64_t bit = i * lb;
    levels[i] = (uint8_t)((lw[bit / 32] >> (bit % 32)) & mask);
  }
}

// ------------------------------- Elias integer code -----------------------------------------
// Writes Elias(k) as '0'/'1' characters; returns its length (buf needs >= 80 bytes).
int oq_elias_string(uint64_t k, char* buf) {
  const std::string s = elias_string(k);
  std::memcpy(buf, s.data(), s.size());
  buf[s.size()] = 0;
  return (int)s.size();
}

// Decodes one integer from a '0'/'1' character string; returns bits consumed, or -1.
int oq_elias_parse(const char* bits, int nbits, uint64_t* value) {
  std::vector<uint32_t> w((size_t)(nbits + 31) / 32 + 1, 0u);
  for (int t = 0; t < nbits; ++t)
    if (bits[t] == '1') w[(size_t)t >> 5] |= (uint32_t)1u << (31 - (t & 31));
  BitReader br{w.data(), 0, (uint64_t)nbits, false};
  const uint64_t v = elias_read(br);
  if (br.fail) return -1;
  *value = v;
  return (int)br.pos;
}

// ------------------------------- Elias-coded messages ---------------------------------------
// Code_s per bucket (Section 3.1): 32 bits of A, then for every nonzero level in index order
// Elias(distance from the previous nonzero; first one: its 1-based position), sign bit,
// Elias(level). Code'_s (dense = 1, Appendix A.3): 32 bits of A, then for EVERY coordinate
// sign bit, Elias(level + 1). Bucket strings are concatenated with no padding; offsets[b] is
// the first bit of bucket b, offsets[B] the payload length. Returns payload bits, or
// (uint64_t)-1 if cap_bytes is too small (payload is then incomplete).
uint64_t oq_elias_pack(const float* A, const uint8_t* levels, const uint8_t* signs, uint64_t n,
                       uint32_t d, int dense, uint8_t* payload, uint64_t cap_bytes,
                       uint64_t* offsets) {
  std::memset(payload, 0, cap_bytes);
  BitWriter bw{(uint32_t*)payload, (cap_bytes / 4) * 32, 0, false};
  const uint64_t B = n_buckets(n, d);
  for (uint64_t b = 0; b < B; ++b) {
    offsets[b] = bw.pos;
    const uint64_t lo = b * d, hi = (lo + d < n) ? lo + d : n;
    const uint32_t abits = float_bits(A[b]);
    for (int t = 31; t >= 0; --t) bw.put((int)((abits >> t) & 1u));
    if (dense) {
      for (uint64_t i = lo; i < hi; ++i) {
        bw.put(signs[i] ? 1 : 0);
        bw.put_str(elias_string((uint64_t)levels[i] + 1));
      }
    } else {
      int64_t prev = -1;
      for (uint64_t i = lo; i < hi; ++i) {
        if (levels[i] == 0) continue;
        const int64_t j = (int64_t)(i - lo);
        bw.put_str(elias_string((uint64_t)(j - prev)));
        bw.put(signs[i] ? 1 : 0);
        bw.put_str(elias_string((uint64_t)levels[i]));
        prev = j;
      }
    }
  }
  offsets[B] = bw.pos;
  return bw.overflow ? (uint64_t)-1 : bw.pos;
}

// Inverse of oq_elias_pack. Returns 0, or a nonzero code for a malformed stream:
// 1 bucket shorter than 32 bits or offsets not ascending, 2 code runs past the bucket's end,
// 3 position outside the bucket, 4 level outside [1, s] (dense: [0, s]).
int oq_elias_unpack(const uint8_t* payload, const uint64_t* offsets, uint64_t n, uint32_t d,
                    uint32_t s, int dense, float* A, uint8_t* levels, uint8_t* signs) {
  const uint64_t B = n_buckets(n, d);
  std::memset(levels, 0, n);
  std::memset(signs, 0, n);
  for (uint64_t b = 0; b < B; ++b) {
    const uint64_t lo = b * d, hi = (lo + d < n) ? lo + d : n;
    if (offsets[b + 1] < offsets[b] || offsets[b + 1] - offsets[b] < 32) return 1;
    BitReader br{(const uint32_t*)payload, offsets[b], offsets[b + 1], false};
    uint32_t abits = 0;
    for (int t = 0; t < 32; ++t) abits = (abits << 1) | (uint32_t)br.get();
    A[b] = bits_float(abits);
    if (dense) {
      for (uint64_t i = lo; i < hi; ++i) {
        const int sg = br.get();
        const uint64_t l1 = elias_read(br);
        if (br.fail) return 2;
        if (l1 < 1 || l1 - 1 > s) return 4;
        levels[i] = (uint8_t)(l1 - 1);
        signs[i] = (uint8_t)sg;
      }
      if (br.pos != br.end) return 2;
    } else {
      int64_t pos = -1;
      while (br.pos < br.end) {
        const uint64_t gap = elias_read(br);
        if (br.fail) return 2;
        pos += (int64_t)gap;
        if (pos < 0 || (uint64_t)pos >= hi - lo) return 3;
        const int sg = br.get();
        const uint64_t l = elias_read(br);
        if (br.fail) return 2;
        if (l < 1 || l > s) return 4;
        levels[lo + (uint64_t)pos] = (uint8_t)l;
        signs[lo + (uint64_t)pos] = (uint8_t)sg;
      }
    }
  }
  return 0;
}

// Worst-case message bytes. Fixed: exact. Elias: 32 bits per bucket plus, per coordinate, the
// longest (gap, sign, level) triple with gap 1, i.e. 2 + |Elias(s)| bits (dense: 1 +
// |Elias(s + 1)|), padded, plus the (B + 1)-entry u64 offset table.
uint64_t oq_message_capacity(uint64_t n, uint32_t d, uint32_t s, int code_kind) {
  if (code_kind == OQ_CODE_FIXED) { uint64_t lay[4]; oq_fixed_layout(n, d, s, lay); return lay[2]; }
  const uint64_t B = n_buckets(n, d);
  const uint64_t per = (code_kind == OQ_CODE_ELIAS)
                           ? 2 + (uint64_t)elias_string(s).size()
                           : 1 + (uint64_t)elias_string((uint64_t)s + 1).size();
  const uint64_t bits = 32 * B + n * per;
  return align16((bits + 7) / 8) + 8 * (B + 1);
}

// ------------------------------- whole-message Encode / Decode ------------------------------
// Encode(g): scales (or A_ext verbatim when not null), levels, message bytes.
// info[0] = payload bits (fixed: 8 * total bytes), info[1] = byte offset of the offset table
// (0 for fixed), info[2] = total message bytes, info[3] = 0.
// Returns 0, or -1 when cap_bytes is too small.
int oq_encode(const float* g, uint64_t n, uint32_t d, uint32_t s, int norm_kind, int code_kind,
              uint64_t seed, uint32_t step, uint32_t worker, const float* A_ext, uint8_t* out,
              uint64_t cap_bytes, uint64_t* info) {
  const uint64_t B = n_buckets(n, d);
  std::vector<float> A(B);
  if (A_ext) std::memcpy(A.data(), A_ext, 4 * B);
  else oq_bucket_scales(g, n, d, norm_kind, A.data());
  std::vector<uint8_t> levels(n), signs(n);
  oq_quantize(g, n, d, s, A.data(), seed, step, worker, 0, levels.data(), signs.data());
  if (code_kind == OQ_CODE_FIXED) {
    uint64_t lay[4];
    oq_fixed_layout(n, d, s, lay);
    if (cap_bytes < lay[2]) return -1;
    oq_fixed_pack(A.data(), levels.data(), signs.data(), n, d, s, out);
    info[0] = 8 * lay[2]; info[1] = 0; info[2] = lay[2]; info[3] = 0;
    return 0;
  }
  std::vector<uint64_t> off(B + 1);
  // First pass into a scratch buffer of worst-case size gives the payload length.
  const uint64_t worst = oq_message_capacity(n, d, s, code_kind);
  std::vector<uint8_t> tmp(worst);
  const uint64_t bits = oq_elias_pack(A.data(), levels.data(), signs.data(), n, d,
                                      code_kind == OQ_CODE_ELIAS_DENSE, tmp.data(), worst,
                                      off.data());
  if (bits == (uint64_t)-1) return -1;
  const uint64_t pay = align16((bits + 7) / 8);
  const uint64_t total = pay + 8 * (B + 1);
  if (cap_bytes < total) return -1;
  std::memcpy(out, tmp.data(), pay);
  std::memcpy(out + pay, off.data(), 8 * (B + 1));
  info[0] = bits; info[1] = pay; info[2] = total; info[3] = 0;
  return 0;
}

// Decode one message into dense Q_s values. table = offsets (Elias kinds), ignored for fixed.
int oq_decode(const uint8_t* msg, const uint64_t* table, uint64_t n, uint32_t d, uint32_t s,
              int code_kind, float* out) {
  const uint64_t B = n_buckets(n, d);
  std::vector<float> A(B);
  std::vector<uint8_t> levels(n), signs(n);
  if (code_kind == OQ_CODE_FIXED) {
    oq_fixed_unpack(msg, n, d, s, A.data(), levels.data(), signs.data());
  } else {
    const int st = oq_elias_unpack(msg, table, n, d, s, code_kind == OQ_CODE_ELIAS_DENSE,
                                   A.data(), levels.data(), signs.data());
    if (st) return st;
  }
  oq_dequantize(A.data(), levels.data(), signs.data(), n, d, s, out);
  return 0;
}

// Algorithm 1, the sum over peers: acc_i = ((+0 + g^0_i) + g^1_i) + ... in ascending k.
int oq_decode_accumulate(const uint8_t* const* msgs, const uint64_t* const* tables, uint32_t K,
                         uint64_t n, uint32_t d, uint32_t s, int code_kind, float* acc) {
  std::vector<float> gk(n);
  for (uint64_t i = 0; i < n; ++i) acc[i] = 0.0f;
  for (uint32_t k = 0; k < K; ++k) {
    const int st = oq_decode(msgs[k], tables ? tables[k] : nullptr, n, d, s, code_kind, gk.data());
    if (st) return st;
    for (uint64_t i = 0; i < n; ++i) acc[i] = acc[i] + gk[i];
  }
  return 0;
}

// Algorithm 1, last line: x <- x - (eta / K) * acc, with c = eta / K formed once.
void oq_sgd_step(float* x, const float* acc, float eta, uint32_t K, uint64_t n) {
  const float c = eta / (float)K;
  for (uint64_t i = 0; i < n; ++i) {
    const float p = c * acc[i];
    x[i] = x[i] - p;
  }
}

}  // extern "C"
