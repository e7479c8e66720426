// Elias decode for shapes the shared-memory decoders do not reach (more than 32 peers with long
// buckets): one warp per bucket, the peers parsed in passes into byte (or 16-bit) codes, summed in
// ascending k. Slow and general.
#include "elias_decode.cuh"

namespace qsgd {

namespace {

constexpr int kWarps = 4;
constexpr int kThreads = kWarps * 32;

template <typename CodeT> struct CodeTraits;
template <> struct CodeTraits<uint8_t> { static constexpr uint32_t kSignBit = 0x80u; };
template <> struct CodeTraits<uint16_t> { static constexpr uint32_t kSignBit = 0x8000u; };

// Parses one bucket string of one peer into codes[0..db). Returns a QSGD_DEV_* mask.
template <typename CodeT, bool DENSE>
__device__ __forceinline__ uint32_t parse_bucket(const PeerSet& peers, uint32_t k, uint64_t b,
                                                 uint64_t B, uint32_t db, uint32_t s,
                                                 CodeT* __restrict__ codes, float* A_out) {
  *A_out = 0.f;
  const StringRef ref = string_ref(peers, k, b, B, db);
  if (ref.err) return ref.err;
  const uint32_t* __restrict__ words = ref.words;
  const uint64_t lo = ref.lo, hi = ref.lo + 32ull + ref.total;
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
  chain_wait();                                   // the messages come from the kernels ahead
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
        const uint32_t st = parse_bucket<CodeT, DENSE>(p.peers, k0 + kk, b, p.B, db, p.s,
                                                       codes + (size_t)kk * p.d, &A);
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
    const cudaError_t le = launch_chained(kern, grid, kThreads, smem, stream, p);
    if (le != cudaSuccess) return (int)le;
  }
  return (int)cudaGetLastError();
}

}  // namespace

int launch_elias_slow(EliasDecodeParams& p, bool dense, bool fused, cudaStream_t stream) {
  if (p.s <= 127) return dense ? launch_slow<uint8_t, true>(p, fused, stream) : launch_slow<uint8_t, false>(p, fused, stream);
  return dense ? launch_slow<uint16_t, true>(p, fused, stream) : launch_slow<uint16_t, false>(p, fused, stream);
}

}  // namespace qsgd
