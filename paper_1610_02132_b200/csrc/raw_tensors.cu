// Raw tensors of the per-tensor policy (Section 5, "Protocol": tensors under a size threshold are
// not quantized). Their fp32 values travel in a region in front of the message proper; Decode adds
// the K regions in ascending k from +0 (the same order as the quantized coordinates) and either
// stores the sums at the tensors' places or applies the SGD step x <- x - (eta / K) * sum there.
// The raw part is tiny next to the quantized part (0.02 % to 0.3 % of the coordinates of the
// AlexNet- and ResNet-152-shaped gradients), so these kernels are one thread per element with a
// binary search over the segment table.
#include "qsgd_common.cuh"

namespace qsgd {

namespace {

constexpr int kThreads = 256;

// Segment that holds raw element j: the largest i with start[i] <= j.
__device__ __forceinline__ uint64_t find_segment(const uint64_t* __restrict__ start, uint64_t R, uint64_t j) {
  uint64_t lo = 0, hi = R;                      // invariant: start[lo] <= j < start[hi]
  while (hi - lo > 1) {
    const uint64_t mid = (lo + hi) >> 1;
    if (__ldg(start + mid) <= j) lo = mid; else hi = mid;
  }
  return lo;
}

__global__ void __launch_bounds__(kThreads) raw_gather_kernel(const float* __restrict__ g, const RawSegments raw,
                                                            float* __restrict__ out_raw, uint64_t padded,
                                                            uint64_t* info, int has_compact) {
  const uint64_t j = (uint64_t)blockIdx.x * kThreads + threadIdx.x;
  chain_wait();
  if (j < raw.n_raw) {
    const uint64_t sgm = find_segment(raw.start, raw.R, j);
    out_raw[j] = g[__ldg(raw.src + sgm) + (j - __ldg(raw.start + sgm))];
  } else if (j < padded) {
    out_raw[j] = 0.f;                            // padding of the region to 16 bytes
  }
  if (j == 0 && info) {
    // message sizes: the encoder of the compact part wrote its own; put the raw region in front
    const uint64_t prefix = 4 * padded;
    if (has_compact) {
      info[0] += 32 * raw.n_raw;
      info[1] = info[1] ? info[1] + prefix : 0;
      info[2] += prefix;
    } else {
      info[0] = 32 * raw.n_raw; info[1] = 0; info[2] = prefix;
    }
    info[3] = prefix;
  }
}

struct RawPeers { const float* region[QSGD_MAX_PEERS]; };

template <bool FUSED>
__global__ void __launch_bounds__(kThreads) raw_decode_kernel(const __grid_constant__ RawPeers peers, uint32_t K,
                                                            const RawSegments raw, float* __restrict__ out, float c) {
  const uint64_t j = (uint64_t)blockIdx.x * kThreads + threadIdx.x;
  chain_wait();
  if (j >= raw.n_raw) return;
  float acc = 0.f;
  for (uint32_t k = 0; k < K; ++k) acc = __fadd_rn(acc, __ldg(peers.region[k] + j));
  const uint64_t sgm = find_segment(raw.start, raw.R, j);
  float* o = out + __ldg(raw.src + sgm) + (j - __ldg(raw.start + sgm));
  *o = FUSED ? __fsub_rn(*o, __fmul_rn(c, acc)) : acc;
}

}  // namespace

int launch_raw_gather(const float* g, const RawSegments& raw, float* out_raw, uint64_t* info, bool has_compact,
                      cudaStream_t stream) {
  const uint64_t padded = (raw.n_raw + 3) & ~3ull;
  const uint64_t threads = padded ? padded : 1;            // one thread at least: it writes the sizes
  const uint32_t grid = (uint32_t)((threads + kThreads - 1) / kThreads);
  {
    ScopedKernel sk(kKernRawGather, stream);
    return (int)launch_chained(raw_gather_kernel, grid, kThreads, 0, stream, g, raw, out_raw, padded, info,
                               has_compact ? 1 : 0);
  }
}

int launch_raw_decode(const float* const* raw_regions, uint32_t K, const RawSegments& raw, float* acc_or_x,
                      bool fused, float eta, cudaStream_t stream) {
  if (raw.n_raw == 0) return 0;
  RawPeers peers;
  for (uint32_t k = 0; k < K; ++k) peers.region[k] = raw_regions[k];
  for (uint32_t k = K; k < QSGD_MAX_PEERS; ++k) peers.region[k] = nullptr;
  const uint32_t grid = (uint32_t)((raw.n_raw + kThreads - 1) / kThreads);
  const float c = eta / (float)K;
  {
    ScopedKernel sk(kKernRawDecode, stream);
    if (fused) return (int)launch_chained(raw_decode_kernel<true>, grid, kThreads, 0, stream, peers, K, raw, acc_or_x, c);
    return (int)launch_chained(raw_decode_kernel<false>, grid, kThreads, 0, stream, peers, K, raw, acc_or_x, c);
  }
}

}  // namespace qsgd
