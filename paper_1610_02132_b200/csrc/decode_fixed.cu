// Decode-and-aggregate, fixed-width path, optionally fused with the SGD step (Algorithm 1:
// g^l <- Decode(M^l); x <- x - (eta / K) * sum_l g^l).
//
// A warp owns chunks of 512 consecutive coordinates, a lane 16 of them, and walks the K
// messages in ascending k, so every coordinate's sum has the fixed order ((0 + g^0) + g^1) ...
// With K = 16 peers there are only a handful of issue slots per (peer, coordinate) at HBM
// speed, so reconstruction A * (level / s) * sign is a table lookup:
//   * s <= 15: the 2 * (s + 1) possible values +-A * (level / s) of one (peer, bucket) live one
//     per lane and are fetched with a warp shuffle indexed by "sign | level"; the sign bits are
//     spread next to the level nibbles with one multiply per four coordinates;
//   * s >= 16: level / s (correctly rounded) comes from a shared-memory table replicated per
//     lane (bank-conflict free), followed by the multiply with A and a sign flip.
#include "decode_common.cuh"

namespace qsgd {

namespace {

constexpr int kThreads = 256;
constexpr int kWarps = kThreads / 32;
constexpr int kChunk = 512;            // coordinates per warp iteration

struct DecodeParams {
  const uint8_t* msg[QSGD_MAX_PEERS];   // the K messages; all share one layout, so the three regions
  uint64_t off_sign, off_level;         // of every message sit at the same byte offsets
  uint32_t K;
  uint64_t n;
  uint32_t d;
  uint32_t s;
  uint32_t log2_chunks_per_bucket;   // valid when single_scale
  float* out;      // acc (overwritten) or x (updated in place)
  float c;         // eta / K (fused only)
  uint64_t chunks;
  BucketMap map;
};

// Peers per unrolled group of the k loop: enough loads in flight to cover their latency, few
// enough that the 16 running sums and the group's words stay in registers (measured per width).
template <int LB> struct PeerUnroll { static constexpr int value = LB == 1 ? 3 : 4; };

template <int LB, bool FUSED, bool SINGLE>
__global__ void __launch_bounds__(kThreads, 4) decode_fixed_kernel(const __grid_constant__ DecodeParams p) {
  __shared__ __align__(16) float xi_tab[LB == 8 ? 256 * 32 : 32];
  const uint32_t tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const float sf = (float)p.s;
  float lut0 = 0.f;                                  // this lane's +-(level / s)
  if (LB == 8) {
    for (uint32_t i = tid; i < 256 * 32; i += kThreads) xi_tab[i] = __fdiv_rn((float)(i >> 5), sf);
    __syncthreads();
  } else {
    const uint32_t level = lane & ((1u << LB) - 1u), neg = (lane >> LB) & 1u;
    const float q = __fdiv_rn((float)level, sf);
    lut0 = neg ? -q : q;
  }
  const uint8_t* tab_lane = reinterpret_cast<const uint8_t*>(xi_tab) + 4 * lane;
  chain_wait();                                      // the messages come from the kernels ahead

  for (uint64_t ch = (uint64_t)blockIdx.x * kWarps + warp; ch < p.chunks; ch += (uint64_t)gridDim.x * kWarps) {
    const uint64_t i0 = ch * kChunk + (uint64_t)lane * 16;       // first coordinate of this lane
    const bool live = i0 < p.n;                                   // lanes past n only help shuffles
    const uint64_t b = SINGLE ? (ch >> p.log2_chunks_per_bucket) : (live ? i0 / p.d : 0);
    float acc[16];
#pragma unroll
    for (int e = 0; e < 16; ++e) acc[e] = 0.f;

    // byte offsets of this lane's scale, 16 sign bits and 16 level fields inside any message
    const uint64_t slot = i0 >> 4;
    const uint64_t off_a = 4ull * b, off_s = p.off_sign + 2ull * slot, off_l = p.off_level + (uint64_t)(2 * LB) * slot;
#pragma unroll PeerUnroll<LB>::value
    for (uint32_t k = 0; k < p.K; ++k) {
      uint32_t w[4] = {0u, 0u, 0u, 0u};
      uint32_t sb = 0;
      float A = 0.f;
      if (live) {
        const uint8_t* m = p.msg[k];
        A = __ldg(reinterpret_cast<const float*>(m + off_a));
        sb = __ldg(reinterpret_cast<const uint16_t*>(m + off_s));
        if (LB == 8) {
          const uint4 t = __ldg(reinterpret_cast<const uint4*>(m + off_l));
          w[0] = t.x; w[1] = t.y; w[2] = t.z; w[3] = t.w;
        } else if (LB == 4) {
          const uint2 t = __ldg(reinterpret_cast<const uint2*>(m + off_l));
          w[0] = t.x; w[1] = t.y;
        } else if (LB == 2) {
          w[0] = __ldg(reinterpret_cast<const uint32_t*>(m + off_l));
        } else {
          w[0] = __ldg(reinterpret_cast<const uint16_t*>(m + off_l));
        }
      }
      if (LB == 8) add_peer_tab(acc, w, sb, tab_lane, A);
      else if (SINGLE) add_peer_lut<LB, true>(acc, w, sb, __fmul_rn(__shfl_sync(0xffffffffu, A, 0), lut0), A);
      else add_peer_lut<LB, false>(acc, w, sb, lut0, A);
    }

    if (!live) continue;
    if (p.map.src) {                                              // per-tensor policy: buckets live elsewhere
      store_span16<FUSED>(out_span(p.out, p.map, b, (uint32_t)(i0 - b * p.d), p.d, p.n, 16u), acc, p.c);
    } else {
      store_lane16<FUSED>(p.out + i0, acc, i0, p.n, p.c);
    }
  }
}

__global__ void __launch_bounds__(kThreads) sgd_step_kernel(float* __restrict__ x,
                                                           const float* __restrict__ acc, float c,
                                                           uint64_t n) {
  const uint64_t i0 = ((uint64_t)blockIdx.x * kThreads + threadIdx.x) * 4;
  chain_wait();
  if (i0 + 4 <= n) {
    const float4 a = __ldcs(reinterpret_cast<const float4*>(acc + i0));
    float4 v = *reinterpret_cast<const float4*>(x + i0);
    v.x = __fsub_rn(v.x, __fmul_rn(c, a.x));
    v.y = __fsub_rn(v.y, __fmul_rn(c, a.y));
    v.z = __fsub_rn(v.z, __fmul_rn(c, a.z));
    v.w = __fsub_rn(v.w, __fmul_rn(c, a.w));
    *reinterpret_cast<float4*>(x + i0) = v;
  } else {
    for (uint64_t i = i0; i < n; ++i) x[i] = __fsub_rn(x[i], __fmul_rn(c, acc[i]));
  }
}

template <int LB, bool FUSED, bool SINGLE>
int launch_one(const DecodeParams& p, cudaStream_t stream) {
  static KernelSite site;
  auto kern = decode_fixed_kernel<LB, FUSED, SINGLE>;
  int sms = 0, occ = 0;
  const int st = site.lookup(kern, kThreads, 0, &sms, &occ);
  if (st) return st;
  const uint64_t want = (p.chunks + kWarps - 1) / kWarps;
  const uint64_t cap = (uint64_t)sms * occ;
  const uint32_t grid = (uint32_t)(want < cap ? want : cap);
  {
    ScopedKernel sk(kKernDecodeFixed, stream);
    const cudaError_t e = launch_chained(kern, grid, kThreads, 0, stream, p);
    if (e != cudaSuccess) return (int)e;
  }
  return (int)cudaGetLastError();
}

template <int LB>
int launch_lb(const DecodeParams& p, bool fused, bool single, cudaStream_t stream) {
  if (fused) return single ? launch_one<LB, true, true>(p, stream) : launch_one<LB, true, false>(p, stream);
  return single ? launch_one<LB, false, true>(p, stream) : launch_one<LB, false, false>(p, stream);
}

}  // namespace

int launch_decode_fixed(const PeerSet& peers, uint32_t K, uint64_t n, uint32_t d, uint32_t s,
                        float* acc_or_x, bool fused, float eta, const BucketMap& map, cudaStream_t stream) {
  DecodeParams p;
  const FixedLayout L = make_fixed_layout(n, d, s);
  for (uint32_t k = 0; k < K; ++k) p.msg[k] = reinterpret_cast<const uint8_t*>(peers.A[k]);   // the scales open a message
  p.off_sign = L.off_sign; p.off_level = L.off_level;
  p.K = K; p.n = n; p.d = d; p.s = s; p.out = acc_or_x; p.map = map;
  p.c = eta / (float)K;
  p.chunks = (n + kChunk - 1) / kChunk;
  // one scale per chunk when the bucket size is 512 * 2^j
  const bool single = d >= (uint32_t)kChunk && (d & (d - 1)) == 0;
  p.log2_chunks_per_bucket = 0;
  for (uint32_t t = d / kChunk; single && t > 1; t >>= 1) ++p.log2_chunks_per_bucket;
  switch (level_bits_for(s)) {
    case 1: return launch_lb<1>(p, fused, single, stream);
    case 2: return launch_lb<2>(p, fused, single, stream);
    case 4: return launch_lb<4>(p, fused, single, stream);
    default: return launch_lb<8>(p, fused, false, stream);
  }
}

int launch_sgd_step(float* x, const float* acc, float eta, uint32_t K, uint64_t n,
                    cudaStream_t stream) {
  const float c = eta / (float)K;
  const uint64_t quads = (n + 3) / 4;
  const uint32_t grid = (uint32_t)((quads + kThreads - 1) / kThreads);
  {
    ScopedKernel sk(kKernSgdStep, stream);
    const cudaError_t e = launch_chained(sgd_step_kernel, grid, kThreads, 0, stream, x, acc, c, n);
    if (e != cudaSuccess) return (int)e;
  }
  return (int)cudaGetLastError();
}

}  // namespace qsgd
