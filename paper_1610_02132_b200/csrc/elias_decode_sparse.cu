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
// Who runs: when the host can read the payload sizes off the pointers it launches this kernel alone
// (check_regime = 0). Otherwise this kernel and a field-rebuilding kernel are launched back to back,
// each evaluates the same predicate on the payload lengths, and exactly one of them does the work.
#include "elias_decode.cuh"

namespace qsgd {

namespace {

template <bool FUSED>
__global__ void __launch_bounds__(256, 2) decode_elias_sparse_kernel(const __grid_constant__ SparseParams p) {
  extern __shared__ __align__(16) uint32_t ssm[];
  __shared__ float xi[256];
  chain_wait();                                   // the messages come from the kernels ahead
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
      const StringRef ref = string_ref(p.peers, pk, b0 + pg, p.B, db);
      st.err = ref.err;
      if (!ref.err) {
        st.total = ref.total;
        st.src.open(ref.words, ref.lo);
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

}  // namespace

// Launches the sparse-regime kernel when the configuration allows one (K <= 32, Code_s); the
// caller then tells the other decoders to stand down when the predicate holds.
int launch_elias_sparse(const PeerSet& peers, uint32_t K, uint64_t n, uint32_t d, uint32_t s, float* out, bool fused,
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
    const cudaError_t le = launch_chained(kern, grid, warps * 32, smem, stream, p);
    if (le != cudaSuccess) return (int)le;
  }
  *launched = true;
  return (int)cudaGetLastError();
}

}  // namespace qsgd
