// Shared device helpers of the QSGD kernels (sm_100a): Philox4x32-10, message layout,
// bit-field helpers and the internal launch interface between the C ABI and the kernels.
#pragma once

#include <cuda_runtime.h>

#include <utility>
#include <stdint.h>

#include <mutex>

#include "../../include/qsgd.h"

namespace qsgd {

// ------------------------------------------------------------------------------------------
// Layout of the fixed-width message (also the intermediate of the Elias encoder).
// ------------------------------------------------------------------------------------------
struct FixedLayout {
  uint64_t n;          // coordinates
  uint32_t d;          // bucket size
  uint32_t lb;         // level bits per coordinate: 1, 2, 4, 8
  uint64_t B;          // buckets
  uint64_t sign_words; // logical u32 words of the sign bitmap
  uint64_t level_words;
  uint64_t off_sign;   // byte offsets of the regions (each 16-byte aligned)
  uint64_t off_level;
  uint64_t total;      // message bytes
};

__host__ __device__ inline uint64_t align16(uint64_t x) { return (x + 15ull) & ~15ull; }

__host__ __device__ inline uint32_t level_bits_for(uint32_t s) {
  return s <= 1 ? 1u : s <= 3 ? 2u : s <= 15 ? 4u : 8u;
}

__host__ __device__ inline FixedLayout make_fixed_layout(uint64_t n, uint32_t d, uint32_t s) {
  FixedLayout L;
  L.n = n; L.d = d; L.lb = level_bits_for(s);
  L.B = (n + d - 1) / d;
  L.sign_words = (n + 31) / 32;
  L.level_words = (n * L.lb + 31) / 32;
  L.off_sign = align16(4 * L.B);
  L.off_level = L.off_sign + align16(4 * L.sign_words);
  L.total = L.off_level + align16(4 * L.level_words);
  return L;
}

// ------------------------------------------------------------------------------------------
// Philox4x32-10 (Salmon et al., SC'11). One call yields the uniforms of four consecutive
// coordinates: counter = (q lo, q hi, step, worker) with q = i / 4, key = (seed lo, seed hi).
// ------------------------------------------------------------------------------------------
struct PhiloxKey { uint32_t k0, k1; };

__device__ __forceinline__ uint4 philox4x32_10(uint32_t c0, uint32_t c1, uint32_t c2, uint32_t c3,
                                               uint32_t k0, uint32_t k1) {
  constexpr uint32_t M0 = 0xD2511F53u, M1 = 0xCD9E8D57u;
  constexpr uint32_t W0 = 0x9E3779B9u, W1 = 0xBB67AE85u;
#pragma unroll
  for (int r = 0; r < 10; ++r) {
    const uint32_t hi0 = __umulhi(M0, c0), lo0 = M0 * c0;
    const uint32_t hi1 = __umulhi(M1, c2), lo1 = M1 * c2;
    c0 = hi1 ^ c1 ^ k0;
    c1 = lo1;
    c2 = hi0 ^ c3 ^ k1;
    c3 = lo0;
    k0 += W0;
    k1 += W1;
  }
  return make_uint4(c0, c1, c2, c3);
}

// Uniform in [0, 1 - 2^-24]: top 24 bits of a Philox word times 2^-24 (exact in fp32).
__device__ __forceinline__ float u01_from_bits(uint32_t x) {
  return __fmul_rn(__uint2float_rn(x >> 8), 5.9604644775390625e-08f);
}

// Level of one coordinate: min(floor((s * |v|) * r + u), s) with r = 1 / A (0 for a zero
// bucket). Two multiplies and one add, each rounded to nearest, no contraction.
__device__ __forceinline__ uint32_t quantize_level(float v, float r, float sf, uint32_t s,
                                                   uint32_t rnd) {
  const float t = __fmul_rn(__fmul_rn(sf, fabsf(v)), r);
  const float c = __fadd_rn(t, u01_from_bits(rnd));
  const uint32_t l = (uint32_t)__float2int_rz(c);
  return min(l, s);
}

// ------------------------------------------------------------------------------------------
// Internal launch interface (host). Each returns a cudaError_t-compatible int.
// ------------------------------------------------------------------------------------------
struct PeerSet {                 // K messages, resolved to region pointers on the host
  const float* A[QSGD_MAX_PEERS];          // fixed: scale arrays
  const uint32_t* sign[QSGD_MAX_PEERS];    // fixed: sign bitmaps
  const uint32_t* level[QSGD_MAX_PEERS];   // fixed: level fields
  const uint32_t* payload[QSGD_MAX_PEERS]; // Elias: payload words
  const uint64_t* table[QSGD_MAX_PEERS];   // Elias: offset tables; packed form: the message's four info words
  uint64_t bound[QSGD_MAX_PEERS];          // Elias: bytes of payload the caller vouches for (0 = not given);
                                           // packed form: bytes readable from the start of the message
  uint32_t packed;                         // Elias: tables are found on the device, at byte info[1] of each message
};

// Per-tensor policy (Section 5, "Protocol"): the coordinates that get quantized form a "compact"
// vector of whole buckets, and bucket b of it lives at elements [src[b], src[b] + len[b]) of the flat
// gradient (len[b] <= d; the rest of the bucket is zero padding that exists nowhere in memory).
// src == nullptr means the ordinary case: the compact vector is the flat array itself.
struct BucketMap {
  const uint64_t* src;     // device, one entry per bucket
  const uint32_t* len;     // device, one entry per bucket
  uint32_t quads;          // nonzero when every src and len is a multiple of 4 (16-byte accesses stay legal)
};

inline BucketMap no_map() { return BucketMap{nullptr, nullptr, 1u}; }

int launch_quantize_fixed(const float* g, uint64_t n, uint32_t d, uint32_t s, int norm_kind,
                          uint64_t seed, uint32_t step, uint32_t worker, uint8_t* out,
                          uint32_t* status_dev, uint64_t* info, uint32_t* clear_word, const BucketMap& map,
                          cudaStream_t stream);

int launch_decode_fixed(const PeerSet& peers, uint32_t K, uint64_t n, uint32_t d, uint32_t s,
                        float* acc_or_x, bool fused, float eta, const BucketMap& map, cudaStream_t stream);

int launch_sgd_step(float* x, const float* acc, float eta, uint32_t K, uint64_t n,
                    cudaStream_t stream);

size_t elias_workspace_bytes(uint64_t n, uint32_t d, uint32_t s);

int launch_elias_encode(const float* g, uint64_t n, uint32_t d, uint32_t s, int norm_kind,
                        bool dense, uint64_t seed, uint32_t step, uint32_t worker, uint8_t* out,
                        size_t out_capacity, uint64_t* out_bits, uint8_t* workspace,
                        uint32_t* status_dev, const BucketMap& map, cudaStream_t stream);

int launch_decode_elias(const PeerSet& peers, uint32_t K, uint64_t n, uint32_t d, uint32_t s,
                        bool dense, float* acc_or_x, bool fused, float eta, uint32_t* status_dev,
                        const BucketMap& map, cudaStream_t stream);

// Raw tensors of the per-tensor policy: segment j holds elements [raw_src[j], raw_src[j] + raw_start[j+1]
// - raw_start[j]) of the flat array and sits at raw_start[j] in a message's raw region.
struct RawSegments {
  const uint64_t* src;     // device, R entries
  const uint64_t* start;   // device, R + 1 entries, start[R] = n_raw
  uint64_t R;
  uint64_t n_raw;
};

// Copies the raw values into the front of a message and moves the message sizes in info[0..3]
// (written by the encoder of the compact part) behind that raw region.
int launch_raw_gather(const float* g, const RawSegments& raw, float* out_raw, uint64_t* info, bool has_compact,
                      cudaStream_t stream);

// Sum of the K raw regions in ascending k from +0, put at the tensors' places in acc, or applied to x.
int launch_raw_decode(const float* const* raw_regions, uint32_t K, const RawSegments& raw, float* acc_or_x,
                      bool fused, float eta, cudaStream_t stream);

// Every kernel launch is bracketed by one of these: it counts the launch and, while kernel
// timing is switched on (qsgd_profile_enable), records a CUDA event before and after it on the
// launching stream.
enum KernelId {
  kKernQuantize = 0, kKernQuantizeTail, kKernDecodeFixed, kKernSgdStep, kKernEliasLength,
  kKernEliasScatter, kKernDecodeElias, kKernDecodeEliasSparse, kKernRawGather, kKernRawDecode, kKernCount
};

// Launch facts of one kernel that belong to a device, not to the process: the opt-in to more than
// 48 KB of dynamic shared memory, the SM count and the resident CTAs per SM. Looked up once per
// device, with that device current, under a lock; one instance per kernel (a function-local static).
constexpr int kMaxDevices = 64;

struct KernelSite {
  std::mutex mu;
  bool ready[kMaxDevices] = {};
  int sms[kMaxDevices] = {};
  int occ[kMaxDevices] = {};

  template <class Kernel>
  int lookup(Kernel kern, int threads, size_t smem, int* sms_out, int* occ_out) {
    int dev = 0;
    cudaError_t e = cudaGetDevice(&dev);
    if (e != cudaSuccess) return (int)e;
    if (dev < 0 || dev >= kMaxDevices) return (int)cudaErrorInvalidDevice;
    std::lock_guard<std::mutex> lk(mu);
    if (!ready[dev]) {
      e = cudaDeviceGetAttribute(&sms[dev], cudaDevAttrMultiProcessorCount, dev);
      if (e != cudaSuccess) return (int)e;
      if (smem > 48 * 1024) {
        e = cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
        if (e != cudaSuccess) return (int)e;
      }
      int o = 0;
      e = cudaOccupancyMaxActiveBlocksPerMultiprocessor(&o, kern, threads, smem);
      if (e != cudaSuccess) return (int)e;
      occ[dev] = o > 0 ? o : 1;
      ready[dev] = true;
    }
    *sms_out = sms[dev];
    *occ_out = occ[dev];
    return 0;
  }
};

// Test hook: bound (in polls) of the waits inside the streaming encoder's main loop.
void set_quantize_poll_limit(uint32_t polls);
uint32_t default_quantize_poll_limit();

// Programmatic dependent launch. Every kernel of the library is launched with programmatic stream
// serialization, so the launch of the next kernel is prepared while the one ahead still runs and its
// CTAs are placed as that kernel's CTAs leave, and it keeps the stream's order itself: it touches no
// global memory before chain_wait(), which returns once the kernel ahead has completed and its
// writes are visible. No kernel releases its dependents early (griddepcontrol.launch_dependents):
// measured, CTAs of a dependent that sit waiting beside running CTAs slow those down (a third on the
// dense-code encode, whose length and scatter kernels run long), while leaving the release to each
// CTA's exit gains 2 us per launch (3 % on back-to-back encodes) and never loses. A kernel launched
// the ordinary way ahead of or behind these keeps the ordinary order.
bool launch_chaining_enabled();
bool set_launch_chaining(bool on);      // returns the previous setting

#ifdef __CUDACC__
__device__ __forceinline__ void chain_wait() { asm volatile("griddepcontrol.wait;" ::: "memory"); }

template <typename... KArgs, typename... Args>
inline cudaError_t launch_chained(void (*kern)(KArgs...), uint32_t grid, uint32_t block, size_t smem,
                                  cudaStream_t stream, Args&&... args) {
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = dim3(grid);
  cfg.blockDim = dim3(block);
  cfg.dynamicSmemBytes = smem;
  cfg.stream = stream;
  cudaLaunchAttribute attr[1];
  attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  attr[0].val.programmaticStreamSerializationAllowed = 1;
  cfg.attrs = attr;
  cfg.numAttrs = launch_chaining_enabled() ? 1 : 0;
  return cudaLaunchKernelEx(&cfg, kern, std::forward<Args>(args)...);
}
#endif

struct ScopedKernel {
  ScopedKernel(KernelId id, cudaStream_t stream);
  ~ScopedKernel();
  KernelId id;
  cudaStream_t stream;
  cudaEvent_t start;
};

}  // namespace qsgd
