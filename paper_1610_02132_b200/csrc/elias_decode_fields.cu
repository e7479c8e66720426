// Decode-and-aggregate, Elias path, optionally fused with the SGD step (Section 3.1, end of
// "Efficient Coding of Gradients": the receiver takes the 32-bit scale off the front of a string and
// then walks the (gap, sign, level) codes; Appendix A.2 for the integer decoder; Algorithm 1 for the
// sum and the step).
//
// A string S can only be parsed front to back, but buckets and peers are independent once the
// per-bucket offset table gives each string's first bit. A warp owns a group of G buckets.
// Phase 1 (parse): lane (g, k) reads peer k's string of bucket g through a 64-bit register
// window (next word prefetched) and rebuilds that peer's *fixed-width fields* -- level fields
// and sign bitmap -- for the bucket in shared memory. Phase 2 (apply): exactly the fixed-width
// decoder's inner loop, reading the fields from shared memory: every lane takes 16 coordinates
// and adds the peers in ascending k, which fixes the summation order however phase 1 was
// scheduled. Shapes whose fields do not fit in shared memory go to the
// decoder of elias_decode_slow.cu.
#include "elias_decode.cuh"

namespace qsgd {

namespace {

// Dense code: the next kDenseBits stream bits usually hold two or three whole (sign, Elias(level + 1))
// symbols (2, 4, 4, 7 bits for levels 0 .. 3). Entry: symbols held (0 .. 3) | their total length << 2 |
// (level | negative << 3) << (6 + 4 j) for symbol j; only levels <= min(s, 7) are listed.
constexpr uint32_t kDenseBits = 10;

__device__ __forceinline__ void fill_dense_lut(uint32_t* lut, uint32_t s) {
  for (uint32_t i = threadIdx.x; i < (1u << kDenseBits); i += blockDim.x) {
    uint32_t w = i << (32 - kDenseBits), used = 0, held = 0, entry = 0;
    while (held < 3u && used + 2u <= kDenseBits) {
      const uint32_t neg = w >> 31;
      uint32_t v, len;
      if (!elias_from_window(w << 1, v, len) || used + 1u + len > kDenseBits || v - 1u > min(s, 7u)) break;
      entry |= ((v - 1u) | (neg << 3)) << (6u + 4u * held);
      w <<= 1u + len;
      used += 1u + len;
      ++held;
    }
    lut[i] = held | (used << 2) | entry;
  }
}

template <int LB, bool DENSE>
__device__ __forceinline__ uint32_t parse_to_fields(const PeerSet& peers, uint32_t k, uint64_t b,
                                                    uint64_t B, uint32_t db, uint32_t d, uint32_t s,
                                                    const uint16_t* lut, const uint32_t* dense_lut,
                                                    uint32_t* __restrict__ row, float* A_out) {
  *A_out = 0.f;
  const StringRef ref = string_ref(peers, k, b, B, db);
  if (ref.err) return ref.err;
  const uint32_t total = ref.total;
  BitSrc src;
  src.open(ref.words, ref.lo);
  *A_out = __uint_as_float(src.take(32));
  uint32_t* srow = row + ((d * LB) >> 5);            // sign bitmap of this peer row
  uint32_t used = 0, err = 0;
  // The row is zero and only this lane writes it, so fields are OR-ed in place.
  if (DENSE) {
    // every coordinate is coded, in order: level and sign words fill up in registers and are stored
    // whole; up to three symbols per table lookup, one by the definition's decoder otherwise
    uint32_t lw = 0u, sg = 0u;
    auto put = [&](uint32_t c, uint32_t level, uint32_t neg) {
      lw |= level << ((c * LB) & 31);
      sg |= (level ? neg : 0u) << (c & 31);
      if ((((c + 1u) * LB) & 31u) == 0u) { row[(c * LB) >> 5] = lw; lw = 0u; }
      if (((c + 1u) & 31u) == 0u) { srow[c >> 5] = sg; sg = 0u; }
    };
    uint32_t c = 0;
    while (c < db) {
      src.refill();
      const uint32_t e = dense_lut[src.hi >> (32 - kDenseBits)];
      const uint32_t held = e & 3u;
      if (held != 0u && c + held <= db) {
        put(c, (e >> 6) & 7u, (e >> 9) & 1u);
        if (held > 1u) put(c + 1u, (e >> 10) & 7u, (e >> 13) & 1u);
        if (held > 2u) put(c + 2u, (e >> 14) & 7u, (e >> 17) & 1u);
        const uint32_t len = (e >> 2) & 15u;
        src.drop(len);
        used += len;
        c += held;
        if (used > total) { err = QSGD_DEV_OVERRUN; break; }
        continue;
      }
      const uint32_t neg = src.hi >> 31;
      uint32_t v, len;
      const bool ok = elias_from_window(src.hi << 1, v, len);
      src.drop(len + 1u);
      used += len + 1u;
      if (!ok || used > total) { err = QSGD_DEV_OVERRUN; break; }
      if (v - 1u > s) { err = QSGD_DEV_LEVEL; break; }
      put(c, v - 1u, neg);
      ++c;
    }
    if (!err) {
      if ((db * LB) & 31u) row[(db * LB) >> 5] = lw;          // a last word that did not fill up
      if (db & 31u) srow[db >> 5] = sg;
      if (used != total) err = QSGD_DEV_OVERRUN;
    }
  } else {
    uint32_t at = 0xFFFFFFFFu;                        // position of the previous nonzero (-1)
    while (used < total) {
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
      if (at >= db || level - 1u >= s || used > total) {     // one rarely taken branch for all three checks
        err = at >= db ? QSGD_DEV_POSITION : 0u;
        err |= level - 1u >= s ? QSGD_DEV_LEVEL : 0u;
        err |= used > total ? QSGD_DEV_OVERRUN : 0u;
        break;
      }
      row[(at * LB) >> 5] |= level << ((at * LB) & 31);
      srow[at >> 5] |= neg << (at & 31);
    }
  }
  return err;
}

template <int LB, bool DENSE, bool FUSED, bool SINGLE>
__global__ void __launch_bounds__(320) decode_elias_fields_kernel(const __grid_constant__ FieldParams p) {
  extern __shared__ __align__(16) uint32_t fsm[];
  __shared__ __align__(16) float xi_tab[LB == 8 ? 256 * 32 : 32];
  __shared__ uint16_t elias_lut[DENSE ? 1u : (1u << kLutBits)];
  __shared__ uint32_t dense_lut[DENSE ? (1u << kDenseBits) : 1u];
  chain_wait();                                   // the messages come from the kernels ahead
  if (!DENSE && p.defer_sparse && sparse_regime(p.peers, p.K, p.B, p.d)) return;
  const uint32_t tid = threadIdx.x, lane = tid & 31, warp = tid >> 5, nwarps = blockDim.x >> 5;
  const float sf = (float)p.s;
  float lut0 = 0.f;
  if (DENSE) fill_dense_lut(dense_lut, p.s);
  else fill_elias_lut(elias_lut);
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
        const uint32_t st = parse_to_fields<LB, DENSE>(p.peers, k, b, p.B, db, p.d,
                                                       p.s, elias_lut, dense_lut, bucket + k * p.row_words, &A);
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
    const cudaError_t le = launch_chained(kern, grid, warps * 32, smem, stream, p);
    if (le != cudaSuccess) return (int)le;
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
  __shared__ uint32_t dense_lut[DENSE ? (1u << kDenseBits) : 1u];
  if (DENSE) fill_dense_lut(dense_lut, p.s);
  chain_wait();                                   // the messages come from the kernels ahead
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
      const StringRef ref = string_ref(p.peers, pk, b0 + pg, p.B, db);
      st.err = ref.err;
      if (!ref.err) {
        st.total = ref.total;
        st.src.open(ref.words, ref.lo);
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
          // every coordinate is coded, in order: level and sign words fill up in registers and are
          // stored whole (the row is zero, and a range starts on a word boundary)
          const uint32_t lim = min(rend, db), cnt = lim > rbeg ? lim - rbeg : 0u;
          uint32_t lw = 0u, sg = 0u;
          auto put = [&](uint32_t pos, uint32_t level, uint32_t neg) {
            lw |= level << ((pos * LB) & 31);
            sg |= (level ? neg : 0u) << (pos & 31);
            if ((((pos + 1u) * LB) & 31u) == 0u) { row[(pos * LB) >> 5] = lw; lw = 0u; }
            if (((pos + 1u) & 31u) == 0u) { srow[pos >> 5] = sg; sg = 0u; }
          };
          uint32_t pos = 0;
          while (pos < cnt && st.err == 0u) {
            st.src.refill();
            const uint32_t e = dense_lut[st.src.hi >> (32 - kDenseBits)];
            const uint32_t held = e & 3u;
            if (held != 0u && pos + held <= cnt) {            // two or three symbols at once (or one)
              put(pos, (e >> 6) & 7u, (e >> 9) & 1u);
              if (held > 1u) put(pos + 1u, (e >> 10) & 7u, (e >> 13) & 1u);
              if (held > 2u) put(pos + 2u, (e >> 14) & 7u, (e >> 17) & 1u);
              const uint32_t len = (e >> 2) & 15u;
              st.src.drop(len);
              st.used += len;
              pos += held;
              if (st.used > st.total) st.err = QSGD_DEV_OVERRUN;
              continue;
            }
            // one symbol by the definition's decoder: a level above 7, or fewer coordinates left
            // in the range than the entry holds
            const uint32_t neg = st.src.hi >> 31;
            uint32_t v, len;
            const bool ok = elias_from_window(st.src.hi << 1, v, len);
            st.src.drop(len + 1u);
            st.used += len + 1u;
            if (!ok || st.used > st.total) st.err = QSGD_DEV_OVERRUN;
            else if (v - 1u > p.s) st.err = QSGD_DEV_LEVEL;
            else put(pos, v - 1u, neg);
            ++pos;
          }
          if (st.err == 0u && cnt) {                        // a last word that did not fill up
            if ((cnt * LB) & 31u) row[(cnt * LB) >> 5] = lw;
            if (cnt & 31u) srow[cnt >> 5] = sg;
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
    const cudaError_t le = launch_chained(kern, grid, warps * 32, smem, stream, p);
    if (le != cudaSuccess) return (int)le;
  }
  *handled = true;
  return (int)cudaGetLastError();
}

// ------------------------------------------------------------------------------------------------
// Byte-code decoder for s <= 15 (every field width up to 4 bits), Code_s, d < 1024, K <= 32. Same two
// phases as above, with three changes that matter because this decoder is bound by shared-memory
// traffic (table lookups, field writes, shuffles):
//   * the parse writes one byte per nonzero coordinate -- level | negative << 4, which is the lane
//     index of +-A * (level / s) in the shuffle table -- with a plain byte store: no read-modify-write
//     of packed fields, and phase 2 feeds the bytes to the shuffles as they are, with no sign bits to
//     merge into level fields;
//   * a bucket is walked in ranges of 256 positions (a lane keeps its place in its string between
//     ranges: bit window, position, one decoded entry that lies past the range), so the rows of one
//     range are what sits in shared memory and twice as many warps are resident;
//   * sign and level come from one lookup in a 256-entry table (the next 8 stream bits), and the
//     per-entry checks are reduced to one comparison: an entry at or past min(range end, bucket
//     length) is held back, and one that no range takes is a position error at the end.
// Rows are kByteRange + 16 bytes apart so that lanes parsing different strings at similar positions
// spread over the banks.
// ------------------------------------------------------------------------------------------------
constexpr uint32_t kRowPad = 16;
constexpr uint32_t kByteRange = 256;

// value | length << 8 of the Elias code that the 12 bits i start with, 0 when none is complete
__device__ __forceinline__ uint32_t elias_table_entry(uint32_t i) {
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
  return ok ? (N | ((used + 1) << 8)) : 0u;
}

template <bool FUSED, bool SINGLE>
__global__ void __launch_bounds__(512) decode_elias_bytes_kernel(const __grid_constant__ FieldParams p) {
  extern __shared__ __align__(16) uint32_t fsm[];
  __shared__ uint16_t elias_lut[1u << kLutBits];
  __shared__ uint16_t level_lut[256];
  chain_wait();                                   // the messages come from the kernels ahead
  if (p.defer_sparse && sparse_regime(p.peers, p.K, p.B, p.d)) return;
  const uint32_t tid = threadIdx.x, lane = tid & 31, warp = tid >> 5, nwarps = blockDim.x >> 5;
  const float sf = (float)p.s;
  fill_elias_lut(elias_lut);
  // sign + level in one lookup: entry i (the next 8 stream bits) = level | negative << 4 | length << 8 when
  // the bits hold a sign and a complete code of a level <= min(s, 15), else 0
  for (uint32_t i = tid; i < 256; i += blockDim.x) {
    const uint32_t e = elias_table_entry((i & 0x7Fu) << 5);
    const uint32_t level = e & 0xFFu, len = e >> 8;
    level_lut[i] = (e && len <= 7u && level <= p.s && level <= 15u) ? (uint16_t)(level | ((i >> 7) << 4) | ((len + 1u) << 8))
                                                                    : (uint16_t)0;
  }
  __syncthreads();
  float lut0;
  {
    const uint32_t level = lane & 15u, neg = lane >> 4;
    const float q = __fdiv_rn((float)level, sf);
    lut0 = neg ? -q : q;
  }
  const uint32_t R = p.range;                                   // positions per range (multiple of 32)
  const uint32_t row_bytes = R + kRowPad;
  const uint32_t rows_bytes = p.G * p.K * row_bytes;            // per warp: G * K rows, then 32 scales
  uint8_t* mine = reinterpret_cast<uint8_t*>(fsm) + (size_t)warp * (rows_bytes + 128u);
  float* scales = reinterpret_cast<float*>(mine + rows_bytes);
  const uint32_t pg = lane / p.Kpad, pk = lane % p.Kpad;      // parse role: bucket in group, peer
  uint8_t* row = mine + (pg * p.K + pk) * row_bytes;           // this lane's row (when it parses)
  const uint64_t groups = (p.B + p.G - 1) / p.G;
  constexpr uint32_t kNone = 0xFFFFFFFFu;

  for (uint64_t grp = (uint64_t)blockIdx.x * nwarps + warp; grp < groups; grp += (uint64_t)gridDim.x * nwarps) {
    const uint64_t b0 = grp * p.G;
    // ---- open this lane's string ---------------------------------------------------------------
    BitSrc src;
    uint32_t used = 0, total = 0, err = 0, at = 0xFFFFFFFFu, pend = kNone, db = 0;
    float A = 0.f;
    if (pg < p.G && b0 + pg < p.B) db = (uint32_t)min((uint64_t)p.d, p.n - (b0 + pg) * p.d);
    const bool parsing = db != 0u && pk < p.K;
    if (parsing) {
      const StringRef ref = string_ref(p.peers, pk, b0 + pg, p.B, db);
      err = ref.err;
      if (!err) {
        total = ref.total;
        src.open(ref.words, ref.lo);
        A = __uint_as_float(src.take(32));
      }
    }
    scales[lane] = A;
    bool readable = parsing && err == 0u;

    for (uint32_t rbeg = 0; rbeg < p.d; rbeg += R) {
      const uint32_t rend = min(rbeg + R, p.d);
      for (uint32_t q = lane; q < (rows_bytes >> 4); q += 32) reinterpret_cast<uint4*>(mine)[q] = make_uint4(0u, 0u, 0u, 0u);
      __syncwarp();
      // ---- phase 1: this lane's nonzeros of the range, one byte each ----------------------------
      if (readable) {
        const uint32_t lim = min(rend, db);                 // entries at or past it wait (or are errors)
        if (pend != kNone && (pend & 0xFFFFu) < lim) {
          row[(pend & 0xFFFFu) - rbeg] = (uint8_t)(pend >> 16);
          pend = kNone;
        }
        if (pend == kNone) {
          while (used < total) {
            src.refill();                                   // >= 33 bits: a table-decoded triple takes <= 20
            uint32_t gap, l1 = 0, code, l2 = 0;
            const uint32_t e1 = elias_lut[src.hi >> (32 - kLutBits)];
            if (e1) {
              gap = e1 & 0xFFu;
              l1 = e1 >> 8;
            } else {
              if (!src.elias(gap, used)) { err = QSGD_DEV_OVERRUN; break; }
              src.refill();
            }
            const uint32_t e2 = level_lut[__funnelshift_lc(src.lo, src.hi, l1) >> 24];
            if (e2) {
              code = e2;                                    // the byte store keeps level | negative << 4
              l2 = e2 >> 8;
            } else {
              src.drop(l1);
              used += l1;
              l1 = 0;
              const uint32_t neg = src.hi >> 31;
              src.drop(1);
              used += 1;
              uint32_t level;
              if (!src.elias(level, used)) { err = QSGD_DEV_OVERRUN; break; }
              if (level - 1u >= p.s) { err = QSGD_DEV_LEVEL; break; }
              code = level | (neg << 4);
            }
            src.drop(l1 + l2);
            used += l1 + l2;
            at += gap;
            if (at >= lim) { pend = at | ((code & 0x1Fu) << 16); break; }     // a later range's, or past the bucket
            row[at - rbeg] = (uint8_t)code;
          }
          if (err) readable = false;
        }
      }
      __syncwarp();
      // ---- phase 2: ascending-k sum; a lane takes 8 coordinates per pass --------------------------
      const uint32_t slots_per_bucket = (rend - rbeg) >> 3;
      const uint32_t total_slots = p.G * slots_per_bucket;
      for (uint32_t s0 = 0; s0 < total_slots; s0 += 32) {
        const uint32_t slot = s0 + lane;
        const uint32_t g = slot / slots_per_bucket, cl = (slot - g * slots_per_bucket) << 3, c = rbeg + cl;
        const uint64_t b = b0 + g;
        const uint64_t i0 = b * p.d + c;
        const bool in_tile = slot < total_slots;               // rows and scales of bucket g exist in the tile
        const bool live = in_tile && b < p.B && i0 < p.n;
        // a lane past the end of its bucket still holds its share of the bucket's shuffle table
        const uint32_t gg = in_tile ? g : 0u;
        const uint8_t* rows = mine + gg * p.K * row_bytes + cl;
        const float* sc = scales + gg * p.Kpad;
        float acc[8];
#pragma unroll
        for (int e = 0; e < 8; ++e) acc[e] = 0.f;
#pragma unroll 4
        for (uint32_t k = 0; k < p.K; ++k) {
          const uint2 cw = in_tile ? *reinterpret_cast<const uint2*>(rows + k * row_bytes) : make_uint2(0u, 0u);
          const float Ak = sc[k];
          const uint32_t w[2] = {cw.x, cw.y};
          if (SINGLE) {
            const float lutk = __fmul_rn(Ak, lut0);            // every lane of this pass is in bucket g
#pragma unroll
            for (int h = 0; h < 2; ++h)
#pragma unroll
              for (int j = 0; j < 4; ++j)
                acc[4 * h + j] = __fadd_rn(acc[4 * h + j], shfl_f(lutk, w[h] >> (8 * j)));
          } else {
#pragma unroll
            for (int h = 0; h < 2; ++h)
#pragma unroll
              for (int j = 0; j < 4; ++j)
                acc[4 * h + j] = __fadd_rn(acc[4 * h + j], __fmul_rn(Ak, shfl_f(lut0, w[h] >> (8 * j))));
          }
        }
        if (live) {
          float* o;
          uint32_t valid;
          if (p.map.src) {
            const OutSpan sp = out_span(p.out, p.map, b, c, p.d, p.n, 8u);
            o = sp.ptr; valid = sp.valid;
          } else {
            o = p.out + i0;
            valid = (uint32_t)min((uint64_t)8u, p.n - i0);
          }
          if (valid == 8u && (reinterpret_cast<uintptr_t>(o) & 15u) == 0) {
#pragma unroll
            for (int j = 0; j < 2; ++j) {
              float4 r = make_float4(acc[4 * j], acc[4 * j + 1], acc[4 * j + 2], acc[4 * j + 3]);
              if (FUSED) {
                const float4 x = *reinterpret_cast<const float4*>(o + 4 * j);
                r.x = __fsub_rn(x.x, __fmul_rn(p.c, r.x)); r.y = __fsub_rn(x.y, __fmul_rn(p.c, r.y));
                r.z = __fsub_rn(x.z, __fmul_rn(p.c, r.z)); r.w = __fsub_rn(x.w, __fmul_rn(p.c, r.w));
              }
              *reinterpret_cast<float4*>(o + 4 * j) = r;
            }
          } else {
#pragma unroll
            for (int e = 0; e < 8; ++e)
              if ((uint32_t)e < valid) o[e] = FUSED ? __fsub_rn(o[e], __fmul_rn(p.c, acc[e])) : acc[e];
          }
        }
      }
      __syncwarp();
    }
    // a string must end exactly where the table says
    // a string must end exactly where the table says, with no entry left over (one that no range took
    // lies past the bucket)
    if (parsing && err == 0u && pend != kNone) err = QSGD_DEV_POSITION;
    if (parsing && err == 0u && used != total) err = QSGD_DEV_OVERRUN;
    if (err) atomicOr(p.status, err);
    __syncwarp();
  }
}

int launch_bytes(FieldParams& p, bool fused, cudaStream_t stream, bool* handled) {
  *handled = false;
  if (p.K > 32u) return 0;
  int dev = 0, max_smem = 0, sms = 0;
  cudaGetDevice(&dev);
  cudaDeviceGetAttribute(&max_smem, cudaDevAttrMaxSharedMemoryPerBlockOptin, dev);
  cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev);
  uint32_t kpad = 1;
  while (kpad < p.K) kpad <<= 1;
  p.Kpad = kpad;
  p.G = 32u / kpad;
  const uint32_t R = p.d <= kByteRange ? p.d : kByteRange;
  p.range = R;
  const size_t per_warp = (size_t)p.G * p.K * (R + kRowPad) + 128u;
  const size_t per_cta = 8192 + 512 + 1024;                     // the two code tables + slack
  const size_t budget = (size_t)max_smem - per_cta;
  const size_t per_sm = 227u << 10;
  int warps = 0, best = 0;
  for (int w = 1; w <= 16; ++w) {
    if ((size_t)w * per_warp > budget) break;
    const int resident = (int)(per_sm / ((size_t)w * per_warp + per_cta)) * w;
    if (resident > best) { best = resident; warps = w; }
  }
  if (warps == 0) return 0;
  const bool single = (p.d & 255u) == 0;                        // every range is 256 long: a pass of 32 lanes x 8 stays inside one bucket
  void (*kern)(FieldParams);
  if (fused) kern = single ? decode_elias_bytes_kernel<true, true> : decode_elias_bytes_kernel<true, false>;
  else kern = single ? decode_elias_bytes_kernel<false, true> : decode_elias_bytes_kernel<false, false>;
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
    const cudaError_t le = launch_chained(kern, grid, warps * 32, smem, stream, p);
    if (le != cudaSuccess) return (int)le;
  }
  *handled = true;
  return (int)cudaGetLastError();
}


template <int LB>
int launch_fields_lb(FieldParams& p, bool dense, bool fused, cudaStream_t stream, bool* handled) {
  if (!dense && LB != 8 && p.d < 1024u && p.K <= 32u) return launch_bytes(p, fused, stream, handled);
  if (p.d >= 1024u && p.K <= 32u)       // long buckets: fields of one range at a time
    return dense ? launch_ranged<LB, true>(p, fused, stream, handled) : launch_ranged<LB, false>(p, fused, stream, handled);
  return dense ? launch_fields<LB, true>(p, fused, stream, handled) : launch_fields<LB, false>(p, fused, stream, handled);
}

}  // namespace

int launch_elias_fields(FieldParams& p, bool dense, bool fused, cudaStream_t stream, bool* handled) {
  switch (level_bits_for(p.s)) {
    case 1: return launch_fields_lb<1>(p, dense, fused, stream, handled);
    case 2: return launch_fields_lb<2>(p, dense, fused, stream, handled);
    case 4: return launch_fields_lb<4>(p, dense, fused, stream, handled);
    default: return launch_fields_lb<8>(p, dense, fused, stream, handled);
  }
}

}  // namespace qsgd
