// Decode-and-aggregate, Elias path, optionally fused with the SGD step (Section 3.1, end of
// "Efficient Coding of Gradients": scale first, then the codes of the nonzeros in index order;
// Appendix A.2 decoder; Algorithm 1 for the sum and the step): the choice among the decoders. Whole-bucket and ranged field rebuilding live in elias_decode_fields.cu, the
// nonzero-driven decoder of the sparse regime in elias_decode_sparse.cu, the general fallback in
// elias_decode_slow.cu; what they share is in elias_decode.cuh.
#include "elias_decode.cuh"

namespace qsgd {

int launch_decode_elias(const PeerSet& peers, uint32_t K, uint64_t n, uint32_t d, uint32_t s,
                        bool dense, float* acc_or_x, bool fused, float eta, uint32_t* status_dev,
                        const BucketMap& map, cudaStream_t stream) {
  // Which decoder? In a message the offset table follows the padded payload, so table - payload is
  // the payload size and the host can evaluate the regime predicate itself (to within the padding)
  // and launch one kernel. With tables kept elsewhere the sizes are only known on the device: both
  // kernels are launched and exactly one does the work. Either decoder is correct on any input;
  // the choice is about speed only.
  const uint64_t B = (n + d - 1) / d;
  bool sizes_known = !dense && K <= 32u && !peers.packed;
  uint64_t payload_bits = 0;
  for (uint32_t k = 0; k < K && sizes_known; ++k) {
    const uint8_t* w = reinterpret_cast<const uint8_t*>(peers.payload[k]);
    const uint8_t* t = reinterpret_cast<const uint8_t*>(peers.table[k]);
    const uint64_t longest = align16((B * 32ull + n * 40ull + 7ull) / 8ull);   // no legal payload is longer
    if (t <= w || (uint64_t)(t - w) > longest) sizes_known = false;
    else payload_bits += 8ull * (uint64_t)(t - w);
  }
  const bool host_sparse = sizes_known && payload_bits < (uint64_t)K * B * (32ull + d / 4u);
  bool sparse = false;
  {
    FieldParams f;
    f.peers = peers; f.K = K; f.n = n; f.d = d; f.s = s;
    f.B = B;
    f.out = acc_or_x; f.c = eta / (float)K; f.status = status_dev; f.map = map;
    bool handled = false;
    int st = 0;
    if (!dense && (host_sparse || !sizes_known))
      st = launch_elias_sparse(peers, K, n, d, s, acc_or_x, fused, f.c, status_dev, !sizes_known, map, stream, &sparse);
    if (st) return st;
    if (sparse && sizes_known) return 0;                    // the host chose the sparse-regime kernel
    f.defer_sparse = sparse ? 1u : 0u;
    st = launch_elias_fields(f, dense, fused, stream, &handled);
    if (handled || st) return st;
  }
  EliasDecodeParams p;
  p.peers = peers; p.K = K; p.Kc = K; p.n = n; p.d = d; p.s = s;
  p.B = (n + d - 1) / d;
  p.out = acc_or_x; p.c = eta / (float)K; p.status = status_dev; p.warp_bytes = 0;
  p.defer_sparse = sparse ? 1u : 0u; p.map = map;
  return launch_elias_slow(p, dense, fused, stream);
}

}  // namespace qsgd
