// Encode, Elias path (Section 3.1 "Efficient Coding of Gradients", string S; Appendix A.3 for
// the dense variant). Pipeline on one stream:
//   1. quantize into the fixed-width layout held in the workspace (quantize_fixed.cu);
//   2. per-bucket string length L_b, one warp per bucket;
//   3. device-wide exclusive scan of L_b -> bit offsets (block sums, scan of sums, downsweep
//      that also writes the offset table into the message);
//   4. zero the payload, then a warp-cooperative scatter writes every bucket's string at its
//      bit offset: lanes own consecutive sub-ranges of the bucket, a warp scan gives each lane
//      its first bit, words shared between lanes or buckets are merged with atomicOr.
#include <mutex>

#include "elias_common.cuh"

namespace qsgd {

namespace {

constexpr int kThreads = 256;
constexpr int kWarps = kThreads / 32;
constexpr int kScanItems = 4;                         // buckets per thread in the scan kernels
constexpr int kScanBlock = kThreads * kScanItems;     // 1024 buckets per CTA

struct Ctrl {                 // control block at the end of the workspace
  uint64_t total_bits;
  uint64_t payload_bytes;
  uint32_t ok;                // 1 when the message fits out_capacity
  uint32_t pad;
};

struct EliasWs {
  uint8_t* fixed;             // fixed-width intermediate
  uint32_t* len;              // L_b
  uint64_t* off;              // offsets (B + 1)
  uint64_t* block_sums;       // per scan CTA
  Ctrl* ctrl;
  size_t bytes;
};

EliasWs carve(uint8_t* ws, uint64_t n, uint32_t d, uint32_t s) {
  const FixedLayout L = make_fixed_layout(n, d, s);
  EliasWs w;
  size_t o = 0;
  w.fixed = ws + o; o += align16(L.total);
  w.len = reinterpret_cast<uint32_t*>(ws + o); o += align16(4 * L.B);
  w.off = reinterpret_cast<uint64_t*>(ws + o); o += align16(8 * (L.B + 1));
  const uint64_t nblk = (L.B + kScanBlock - 1) / kScanBlock;
  w.block_sums = reinterpret_cast<uint64_t*>(ws + o); o += align16(8 * (nblk + 1));
  w.ctrl = reinterpret_cast<Ctrl*>(ws + o); o += align16(sizeof(Ctrl));
  w.bytes = o;
  return w;
}

// Level field of global coordinate i.
template <int LB>
__device__ __forceinline__ uint32_t level_at(const uint32_t* __restrict__ lw, uint64_t i) {
  const uint64_t bit = i * LB;
  return (__ldg(lw + (bit >> 5)) >> (bit & 31)) & ((1u << LB) - 1u);
}

// Walks the nonzero levels of bucket-relative coordinates [c_lo, c_hi) in index order and
// calls visit(position, level). Whole zero words are skipped.
template <int LB, typename F>
__device__ __forceinline__ void for_each_nonzero(const uint32_t* __restrict__ lw, uint64_t base,
                                                 uint32_t c_lo, uint32_t c_hi, F&& visit) {
  constexpr uint32_t kMask = (1u << LB) - 1u;
  uint32_t c = c_lo;
  while (c < c_hi) {
    const uint64_t bit = (base + c) * LB;
    const uint32_t sh = (uint32_t)(bit & 31);
    uint32_t w = __ldg(lw + (bit >> 5)) >> sh;
    const uint32_t fields = (32u - sh) / LB;
    const uint32_t cnt = min(fields, c_hi - c);
    if (cnt * LB < 32u) w &= (1u << (cnt * LB)) - 1u;
    while (w) {
      const uint32_t f = (uint32_t)(__ffs((int)w) - 1) / LB;
      const uint32_t level = (w >> (f * LB)) & kMask;
      visit(c + f, level);
      w &= ~(kMask << (f * LB));
    }
    c += cnt;
  }
}

struct LaneSummary {
  uint32_t bits;      // bits of this lane's codes, excluding the gap code of its first nonzero
  int32_t first;      // first nonzero position in the lane's range, -1 if none
  int32_t last;       // last nonzero position, -1 if none
};

template <int LB>
__device__ __forceinline__ LaneSummary summarize_sparse(const uint32_t* __restrict__ lw,
                                                        uint64_t base, uint32_t c_lo,
                                                        uint32_t c_hi) {
  LaneSummary s{0u, -1, -1};
  for_each_nonzero<LB>(lw, base, c_lo, c_hi, [&](uint32_t pos, uint32_t level) {
    if (s.first < 0) s.first = (int32_t)pos;
    else s.bits += elias_len(pos - (uint32_t)s.last);
    s.bits += 1u + elias_len(level);
    s.last = (int32_t)pos;
  });
  return s;
}

template <int LB>
__device__ __forceinline__ uint32_t summarize_dense(const uint32_t* __restrict__ lw, uint64_t base,
                                                    uint32_t c_lo, uint32_t c_hi) {
  uint32_t bits = 0;
  for (uint32_t c = c_lo; c < c_hi; ++c) bits += 1u + elias_len(level_at<LB>(lw, base + c) + 1u);
  return bits;
}

// Position of the last nonzero in the lanes before this one (-1 if none).
__device__ __forceinline__ int32_t prev_nonzero_before_lane(int32_t last, uint32_t lane) {
  int32_t run = last;                           // inclusive max-scan of `last`
#pragma unroll
  for (int o = 1; o < 32; o <<= 1) {
    const int32_t t = __shfl_up_sync(0xffffffffu, run, o);
    if (lane >= (uint32_t)o) run = max(run, t);
  }
  const int32_t excl = __shfl_up_sync(0xffffffffu, run, 1);
  return lane == 0 ? -1 : excl;
}

struct BucketParams {
  const float* A;
  const uint32_t* sign;
  const uint32_t* level;
  uint64_t n;
  uint32_t d;
  uint64_t B;
};

// ---- 2. string length per bucket -------------------------------------------------------------
template <int LB, bool DENSE>
__global__ void __launch_bounds__(kThreads) elias_length_kernel(const BucketParams p,
                                                                uint32_t* __restrict__ len) {
  const uint32_t lane = threadIdx.x & 31;
  const uint64_t b = (uint64_t)blockIdx.x * kWarps + (threadIdx.x >> 5);
  if (b >= p.B) return;
  const uint64_t base = b * p.d;
  const uint32_t db = (uint32_t)min((uint64_t)p.d, p.n - base);
  const uint32_t seg = p.d >> 5;
  const uint32_t c_lo = min(lane * seg, db), c_hi = min(c_lo + seg, db);
  uint32_t bits;
  if (DENSE) {
    bits = summarize_dense<LB>(p.level, base, c_lo, c_hi);
  } else {
    const LaneSummary s = summarize_sparse<LB>(p.level, base, c_lo, c_hi);
    const int32_t prev = prev_nonzero_before_lane(s.last, lane);
    bits = s.bits + (s.first >= 0 ? elias_len((uint32_t)(s.first - prev)) : 0u);
  }
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) bits += __shfl_xor_sync(0xffffffffu, bits, o);
  if (lane == 0) len[b] = 32u + bits;
}

// ---- 3. exclusive scan of the lengths --------------------------------------------------------
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

// Message geometry once the payload length is known; capacity check.
__device__ __forceinline__ void finish_totals(uint64_t bits, uint64_t B, size_t out_capacity, Ctrl* ctrl,
                                              uint64_t* __restrict__ out_bits,
                                              uint32_t* __restrict__ status_dev) {
  const uint64_t pay = align16((bits + 7) / 8);
  const uint64_t total_bytes = pay + 8 * (B + 1);
  const bool ok = total_bytes <= out_capacity;
  ctrl->total_bits = bits;
  ctrl->payload_bytes = pay;
  ctrl->ok = ok ? 1u : 0u;
  out_bits[0] = bits; out_bits[1] = pay; out_bits[2] = total_bytes; out_bits[3] = 0;
  if (!ok) atomicOr(status_dev, QSGD_DEV_CAPACITY);
}

// Publishes one bucket offset: workspace copy, table entry, and a zero in the payload word that
// this bucket shares with its predecessor (the scatter ORs into such words, and stores all
// others plainly, so nothing else of the payload needs clearing).
__device__ __forceinline__ void publish_offset(uint64_t b, uint64_t B, uint64_t run, uint32_t len,
                                               bool ok, uint64_t payload_bytes,
                                               uint64_t* __restrict__ off, uint64_t* __restrict__ table,
                                               uint32_t* __restrict__ words) {
  off[b] = run;
  if (ok) {
    table[b] = run;
    if (run & 31) words[run >> 5] = 0u;
  }
  if (b == B - 1) {
    const uint64_t end = run + len;
    off[B] = end;
    if (ok) {
      table[B] = end;
      for (uint64_t w = end >> 5; w < payload_bytes / 4; ++w) words[w] = 0u;   // tail word + padding
    }
  }
}

__global__ void __launch_bounds__(kThreads) scan_block_sums_kernel(const uint32_t* __restrict__ len,
                                                                   uint64_t B,
                                                                   uint64_t* __restrict__ sums) {
  const uint64_t i0 = (uint64_t)blockIdx.x * kScanBlock + threadIdx.x * kScanItems;
  uint64_t v = 0;
#pragma unroll
  for (int j = 0; j < kScanItems; ++j) if (i0 + j < B) v += len[i0 + j];
  uint64_t total;
  block_exclusive_scan(v, &total);
  if (threadIdx.x == 0) sums[blockIdx.x] = total;
}

// One CTA: exclusive scan of the block sums in place; total, message size and capacity check.
__global__ void __launch_bounds__(kThreads) scan_sums_kernel(uint64_t* __restrict__ sums,
                                                             uint64_t nblk, uint64_t B,
                                                             size_t out_capacity, Ctrl* ctrl,
                                                             uint64_t* __restrict__ out_bits,
                                                             uint32_t* __restrict__ status_dev) {
  __shared__ uint64_t carry_s;
  if (threadIdx.x == 0) carry_s = 0;
  __syncthreads();
  for (uint64_t base = 0; base < nblk; base += kThreads) {
    const uint64_t i = base + threadIdx.x;
    const uint64_t v = i < nblk ? sums[i] : 0;
    uint64_t total;
    const uint64_t ex = block_exclusive_scan(v, &total);
    const uint64_t carry = carry_s;
    if (i < nblk) sums[i] = carry + ex;
    __syncthreads();
    if (threadIdx.x == 0) carry_s = carry + total;
    __syncthreads();
  }
  if (threadIdx.x == 0) finish_totals(carry_s, B, out_capacity, ctrl, out_bits, status_dev);
}

__global__ void __launch_bounds__(kThreads) scan_downsweep_kernel(const uint32_t* __restrict__ len,
                                                                  uint64_t B,
                                                                  const uint64_t* __restrict__ sums,
                                                                  const Ctrl* __restrict__ ctrl,
                                                                  uint64_t* __restrict__ off,
                                                                  uint8_t* __restrict__ out) {
  const uint64_t i0 = (uint64_t)blockIdx.x * kScanBlock + threadIdx.x * kScanItems;
  uint32_t l[kScanItems];
  uint64_t v = 0;
#pragma unroll
  for (int j = 0; j < kScanItems; ++j) { l[j] = (i0 + j < B) ? len[i0 + j] : 0u; v += l[j]; }
  uint64_t total;
  uint64_t run = sums[blockIdx.x] + block_exclusive_scan(v, &total);
  const bool ok = ctrl->ok != 0;
  const uint64_t pay = ctrl->payload_bytes;
  uint64_t* table = reinterpret_cast<uint64_t*>(out + pay);
#pragma unroll
  for (int j = 0; j < kScanItems; ++j) {
    if (i0 + j < B) {
      publish_offset(i0 + j, B, run, l[j], ok, pay, off, table, reinterpret_cast<uint32_t*>(out));
      run += l[j];
    }
  }
}

// Whole scan in one CTA of 1024 threads, for messages with few buckets (saves two launches).
constexpr int kSmallScanThreads = 1024;
constexpr uint64_t kSmallScanMaxBuckets = 32768;

__global__ void __launch_bounds__(kSmallScanThreads) scan_small_kernel(
    const uint32_t* __restrict__ len, uint64_t B, size_t out_capacity, Ctrl* ctrl,
    uint64_t* __restrict__ out_bits, uint32_t* __restrict__ status_dev, uint64_t* __restrict__ off,
    uint8_t* __restrict__ out) {
  __shared__ uint64_t carry_s;
  // pass 1: payload length
  uint64_t mine = 0;
  for (uint64_t i = threadIdx.x; i < B; i += kSmallScanThreads) mine += len[i];
  uint64_t total;
  block_exclusive_scan(mine, &total);
  if (threadIdx.x == 0) {
    finish_totals(total, B, out_capacity, ctrl, out_bits, status_dev);
    carry_s = 0;
  }
  __syncthreads();
  const bool ok = ctrl->ok != 0;
  const uint64_t pay = ctrl->payload_bytes;
  uint64_t* table = reinterpret_cast<uint64_t*>(out + pay);
  // pass 2: offsets
  for (uint64_t base = 0; base < B; base += kSmallScanThreads) {
    const uint64_t i = base + threadIdx.x;
    const uint32_t l = i < B ? len[i] : 0u;
    uint64_t chunk;
    const uint64_t ex = block_exclusive_scan(l, &chunk);
    const uint64_t carry = carry_s;
    if (i < B) publish_offset(i, B, carry + ex, l, ok, pay, off, table, reinterpret_cast<uint32_t*>(out));
    __syncthreads();
    if (threadIdx.x == 0) carry_s = carry + chunk;
    __syncthreads();
  }
}

// ---- 4. scatter ----------------------------------------------------------------------------------
// Lane-private writer into the warp's staging words in shared memory (bits of neighbouring lanes
// meet inside a word, so words are OR-ed atomically; shared-memory atomics are cheap).
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
                                                                 const uint64_t* __restrict__ off,
                                                                 const Ctrl* __restrict__ ctrl,
                                                                 uint8_t* __restrict__ out,
                                                                 uint32_t stage_words) {
  extern __shared__ uint32_t stage_all[];
  if (!ctrl->ok) return;
  const uint32_t lane = threadIdx.x & 31;
  uint32_t* stage = stage_all + (size_t)(threadIdx.x >> 5) * stage_words;
  const uint64_t b = (uint64_t)blockIdx.x * kWarps + (threadIdx.x >> 5);
  if (b >= p.B) return;
  const uint64_t base = b * p.d;
  const uint32_t db = (uint32_t)min((uint64_t)p.d, p.n - base);
  const uint32_t seg = p.d >> 5;
  const uint32_t c_lo = min(lane * seg, db), c_hi = min(c_lo + seg, db);
  const uint64_t o0 = __ldg(off + b), o1 = __ldg(off + b + 1);
  const uint32_t lead = (uint32_t)(o0 & 31);                       // bits of the first word owned by b - 1
  const uint32_t nwords = (uint32_t)((lead + (o1 - o0) + 31) >> 5); // words this bucket touches
  for (uint32_t j = lane; j < nwords; j += 32) stage[j] = 0u;

  uint32_t bits;
  int32_t prev = -1;
  if (DENSE) {
    bits = summarize_dense<LB>(p.level, base, c_lo, c_hi);
  } else {
    const LaneSummary s = summarize_sparse<LB>(p.level, base, c_lo, c_hi);
    prev = prev_nonzero_before_lane(s.last, lane);
    bits = s.bits + (s.first >= 0 ? elias_len((uint32_t)(s.first - prev)) : 0u);
  }
  if (lane == 0) bits += 32u;                       // the scale travels with lane 0
  uint32_t inc = bits;
#pragma unroll
  for (int o = 1; o < 32; o <<= 1) {
    const uint32_t t = __shfl_up_sync(0xffffffffu, inc, o);
    if (lane >= (uint32_t)o) inc += t;
  }
  __syncwarp();                                     // staging is zeroed
  if (bits != 0) {
    StageWriter bw;
    bw.begin(stage, lead + (inc - bits));
    if (lane == 0) bw.put(__float_as_uint(__ldg(p.A + b)), 32);
    if (DENSE) {
      for (uint32_t c = c_lo; c < c_hi; ++c) {
        const uint64_t i = base + c;
        const uint32_t sg = (__ldg(p.sign + (i >> 5)) >> (i & 31)) & 1u;
        uint32_t ln;
        const uint32_t code = elias_code(level_at<LB>(p.level, i) + 1u, &ln);
        bw.put((sg << ln) | code, ln + 1);
      }
    } else {
      for_each_nonzero<LB>(p.level, base, c_lo, c_hi, [&](uint32_t pos, uint32_t level) {
        uint32_t ln;
        uint32_t code = elias_code(pos - (uint32_t)prev, &ln);
        bw.put(code, ln);
        const uint64_t i = base + pos;
        const uint32_t sg = (__ldg(p.sign + (i >> 5)) >> (i & 31)) & 1u;
        code = elias_code(level, &ln);
        bw.put((sg << ln) | code, ln + 1);
        prev = (int32_t)pos;
      });
    }
    bw.finish();
  }
  __syncwarp();
  // flush: words owned by this bucket alone are stored, words shared with a neighbour are OR-ed
  uint32_t* gw = reinterpret_cast<uint32_t*>(out) + (o0 >> 5);
  const bool last_shared = ((lead + (o1 - o0)) & 31) != 0;
  for (uint32_t j = lane; j < nwords; j += 32) {
    const uint32_t v = stage[j];
    const bool shared = (j == 0 && lead != 0) || (j == nwords - 1 && last_shared);
    if (shared) atomicOr(gw + j, v);
    else gw[j] = v;
  }
}

template <int LB, bool DENSE>
int run_pipeline(const BucketParams& bp, const EliasWs& w, uint32_t s, uint8_t* out, size_t out_capacity,
                 uint64_t* out_bits, uint32_t* status_dev, cudaStream_t stream) {
  const uint32_t bucket_grid = (uint32_t)((bp.B + kWarps - 1) / kWarps);
  const uint64_t nblk = (bp.B + kScanBlock - 1) / kScanBlock;
  {
    ScopedKernel sk(kKernEliasLength, stream);
    elias_length_kernel<LB, DENSE><<<bucket_grid, kThreads, 0, stream>>>(bp, w.len);
  }
  if (bp.B <= kSmallScanMaxBuckets) {
    ScopedKernel sk(kKernScanSums, stream);
    scan_small_kernel<<<1, kSmallScanThreads, 0, stream>>>(w.len, bp.B, out_capacity, w.ctrl, out_bits,
                                                           status_dev, w.off, out);
  } else {
    {
      ScopedKernel sk(kKernScanBlockSums, stream);
      scan_block_sums_kernel<<<(uint32_t)nblk, kThreads, 0, stream>>>(w.len, bp.B, w.block_sums);
    }
    {
      ScopedKernel sk(kKernScanSums, stream);
      scan_sums_kernel<<<1, kThreads, 0, stream>>>(w.block_sums, nblk, bp.B, out_capacity, w.ctrl,
                                                   out_bits, status_dev);
    }
    {
      ScopedKernel sk(kKernScanDownsweep, stream);
      scan_downsweep_kernel<<<(uint32_t)nblk, kThreads, 0, stream>>>(w.len, bp.B, w.block_sums,
                                                                     w.ctrl, w.off, out);
    }
  }
  {
    // staging: the longest legal string of one bucket, plus the shared lead-in word
    uint32_t elen_max = 1;
    for (uint32_t k = DENSE ? s + 1 : s; k > 1;) { uint32_t m = 0; for (uint32_t t = k; t; t >>= 1) ++m; elen_max += m; k = m - 1; }
    const uint32_t per = DENSE ? 1 + elen_max : 2 + elen_max;
    const uint32_t stage_words = ((32 + bp.d * per + 31) / 32 + 2 + 3) & ~3u;
    const size_t smem = (size_t)stage_words * 4 * kWarps;
    auto kern = elias_scatter_kernel<LB, DENSE>;
    if (smem > 48 * 1024) {
      cudaError_t e = cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
      if (e != cudaSuccess) return (int)e;
    }
    ScopedKernel sk(kKernEliasScatter, stream);
    kern<<<bucket_grid, kThreads, smem, stream>>>(bp, w.off, w.ctrl, out, stage_words);
  }
  return (int)cudaGetLastError();
}

}  // namespace

size_t elias_workspace_bytes(uint64_t n, uint32_t d, uint32_t s) {
  return carve(nullptr, n, d, s).bytes;
}

int launch_elias_encode(const float* g, uint64_t n, uint32_t d, uint32_t s, int norm_kind,
                        bool dense, uint64_t seed, uint32_t step, uint32_t worker, uint8_t* out,
                        size_t out_capacity, uint64_t* out_bits, uint8_t* workspace,
                        uint32_t* status_dev, cudaStream_t stream) {
  const EliasWs w = carve(workspace, n, d, s);
  int st = launch_quantize_fixed(g, n, d, s, norm_kind, seed, step, worker, w.fixed, status_dev, nullptr, stream);
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
  if (n == 0) return QSGD_ERR_SIZE;
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
                             status_dev, static_cast<cudaStream_t>(stream));
}

}  // extern "C"
