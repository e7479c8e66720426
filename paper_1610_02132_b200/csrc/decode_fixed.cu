// Decode-and-aggregate, fixed-width path, optionally fused with the SGD step (Algorithm 1:
// g^l <- Decode(M^l); x <- x - (eta / K) * sum_l g^l). A thread owns 8 consecutive
// coordinates and walks the K messages in ascending k, so every coordinate's sum has the fixed
// order ((0 + g^0) + g^1) + ... . Reconstruction is A * (level / s): level / s comes from a
// table of correctly rounded quotients, then one multiply (Eq. 2).
#include "qsgd_common.cuh"

namespace qsgd {

namespace {

constexpr int kThreads = 256;

struct DecodeParams {
  PeerSet peers;
  uint32_t K;
  uint64_t n;
  uint32_t d;
  uint32_t s;
  float* out;      // acc (overwritten) or x (updated in place)
  float c;         // eta / K (fused only)
};

template <int LB, bool FUSED>
__global__ void __launch_bounds__(kThreads) decode_fixed_kernel(const __grid_constant__ DecodeParams p) {
  __shared__ float xi[256];
  const float sf = (float)p.s;
  for (uint32_t l = threadIdx.x; l < (1u << LB); l += kThreads) xi[l] = __fdiv_rn((float)l, sf);
  __syncthreads();

  const uint64_t grp = (uint64_t)blockIdx.x * kThreads + threadIdx.x;
  const uint64_t i0 = grp * 8;
  if (i0 >= p.n) return;
  const uint64_t b = i0 / p.d;
  constexpr uint32_t kMask = (1u << LB) - 1u;

  float acc[8];
#pragma unroll
  for (int e = 0; e < 8; ++e) acc[e] = 0.f;

  for (uint32_t k = 0; k < p.K; ++k) {
    const float A = __ldg(p.peers.A[k] + b);
    const uint32_t sb = __ldg(reinterpret_cast<const uint8_t*>(p.peers.sign[k]) + grp);
    uint32_t w0, w1 = 0;
    if (LB == 8) {
      const uint2 t = __ldg(reinterpret_cast<const uint2*>(p.peers.level[k]) + grp);
      w0 = t.x; w1 = t.y;
    } else if (LB == 4) {
      w0 = __ldg(p.peers.level[k] + grp);
    } else if (LB == 2) {
      w0 = __ldg(reinterpret_cast<const uint16_t*>(p.peers.level[k]) + grp);
    } else {
      w0 = __ldg(reinterpret_cast<const uint8_t*>(p.peers.level[k]) + grp);
    }
#pragma unroll
    for (int e = 0; e < 8; ++e) {
      uint32_t l;
      if (LB == 8) l = ((e < 4 ? w0 : w1) >> (8 * (e & 3))) & 0xFFu;
      else l = (w0 >> (LB * e)) & kMask;
      float m = __fmul_rn(A, xi[l]);
      if ((sb >> e) & 1u) m = -m;
      acc[e] = __fadd_rn(acc[e], m);
    }
  }

  float* o = p.out + i0;
  if (i0 + 8 <= p.n) {
    float4 r0, r1;
    if (FUSED) {
      const float4 x0 = *reinterpret_cast<const float4*>(o);
      const float4 x1 = *reinterpret_cast<const float4*>(o + 4);
      r0.x = __fsub_rn(x0.x, __fmul_rn(p.c, acc[0])); r0.y = __fsub_rn(x0.y, __fmul_rn(p.c, acc[1]));
      r0.z = __fsub_rn(x0.z, __fmul_rn(p.c, acc[2])); r0.w = __fsub_rn(x0.w, __fmul_rn(p.c, acc[3]));
      r1.x = __fsub_rn(x1.x, __fmul_rn(p.c, acc[4])); r1.y = __fsub_rn(x1.y, __fmul_rn(p.c, acc[5]));
      r1.z = __fsub_rn(x1.z, __fmul_rn(p.c, acc[6])); r1.w = __fsub_rn(x1.w, __fmul_rn(p.c, acc[7]));
    } else {
      r0 = make_float4(acc[0], acc[1], acc[2], acc[3]);
      r1 = make_float4(acc[4], acc[5], acc[6], acc[7]);
    }
    *reinterpret_cast<float4*>(o) = r0;
    *reinterpret_cast<float4*>(o + 4) = r1;
  } else {
#pragma unroll
    for (int e = 0; e < 8; ++e) {
      if (i0 + e < p.n) o[e] = FUSED ? __fsub_rn(o[e], __fmul_rn(p.c, acc[e])) : acc[e];
    }
  }
}

__global__ void __launch_bounds__(kThreads) sgd_step_kernel(float* __restrict__ x,
                                                           const float* __restrict__ acc, float c,
                                                           uint64_t n) {
  const uint64_t i0 = ((uint64_t)blockIdx.x * kThreads + threadIdx.x) * 4;
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

template <int LB>
int launch_lb(const DecodeParams& p, bool fused, uint32_t grid, cudaStream_t stream) {
  {
    ScopedKernel sk(kKernDecodeFixed, stream);
    if (fused) decode_fixed_kernel<LB, true><<<grid, kThreads, 0, stream>>>(p);
    else decode_fixed_kernel<LB, false><<<grid, kThreads, 0, stream>>>(p);
  }
  return (int)cudaGetLastError();
}

}  // namespace

int launch_decode_fixed(const PeerSet& peers, uint32_t K, uint64_t n, uint32_t d, uint32_t s,
                        float* acc_or_x, bool fused, float eta, cudaStream_t stream) {
  DecodeParams p;
  p.peers = peers; p.K = K; p.n = n; p.d = d; p.s = s; p.out = acc_or_x;
  p.c = eta / (float)K;
  const uint64_t groups = (n + 7) / 8;
  const uint32_t grid = (uint32_t)((groups + kThreads - 1) / kThreads);
  switch (level_bits_for(s)) {
    case 1: return launch_lb<1>(p, fused, grid, stream);
    case 2: return launch_lb<2>(p, fused, grid, stream);
    case 4: return launch_lb<4>(p, fused, grid, stream);
    default: return launch_lb<8>(p, fused, grid, stream);
  }
}

int launch_sgd_step(float* x, const float* acc, float eta, uint32_t K, uint64_t n,
                    cudaStream_t stream) {
  const float c = eta / (float)K;
  const uint64_t quads = (n + 3) / 4;
  const uint32_t grid = (uint32_t)((quads + kThreads - 1) / kThreads);
  {
    ScopedKernel sk(kKernSgdStep, stream);
    sgd_step_kernel<<<grid, kThreads, 0, stream>>>(x, acc, c, n);
  }
  return (int)cudaGetLastError();
}

}  // namespace qsgd
