// C ABI of the QSGD codec: argument validation and dispatch to the kernels. See include/qsgd.h
// for the contract of every entry point.
#include <atomic>
#include <mutex>
#include <vector>

#include "qsgd_common.cuh"

namespace qsgd {

static std::atomic<uint64_t> g_launches{0};
static std::atomic<bool> g_chaining{true};

bool launch_chaining_enabled() { return g_chaining.load(std::memory_order_relaxed); }
bool set_launch_chaining(bool on) { return g_chaining.exchange(on, std::memory_order_relaxed); }
static std::atomic<int> g_profile{0};
static std::mutex g_prof_mu;
struct TimedLaunch { KernelId id; cudaEvent_t a, b; };
static std::vector<TimedLaunch> g_timed;

ScopedKernel::ScopedKernel(KernelId id_, cudaStream_t stream_) : id(id_), stream(stream_), start(nullptr) {
  g_launches.fetch_add(1, std::memory_order_relaxed);
  if (g_profile.load(std::memory_order_relaxed)) {
    cudaEventCreate(&start);
    cudaEventRecord(start, stream);
  }
}

ScopedKernel::~ScopedKernel() {
  if (start) {
    cudaEvent_t stop;
    cudaEventCreate(&stop);
    cudaEventRecord(stop, stream);
    std::lock_guard<std::mutex> lk(g_prof_mu);
    g_timed.push_back({id, start, stop});
  }
}

static const char* const kKernelNames[kKernCount] = {
    "quantize_fixed", "quantize_tail", "decode_fixed", "sgd_step", "elias_length",
    "elias_scatter", "decode_elias", "decode_elias_sparse", "raw_gather", "raw_decode"};

namespace {

inline bool aligned16(const void* p) { return (reinterpret_cast<uintptr_t>(p) & 15u) == 0; }

int check_shape(uint64_t n, uint32_t bucket, uint32_t s, int code_kind) {
  if (n == 0 || n > QSGD_MAX_COORDS) return QSGD_ERR_SIZE;
  if (bucket < 32 || bucket > QSGD_MAX_BUCKET || (bucket & 31u)) return QSGD_ERR_BUCKET;
  if (s < 1 || s > QSGD_MAX_LEVELS) return QSGD_ERR_LEVELS;
  if (code_kind != QSGD_CODE_FIXED && code_kind != QSGD_CODE_ELIAS && code_kind != QSGD_CODE_ELIAS_DENSE)
    return QSGD_ERR_KIND;
  return QSGD_OK;
}

// |Elias(k)| on the host, from the recursive definition (Appendix A.2).
uint32_t host_elias_len(uint32_t k) {
  uint32_t len = 1;
  while (k > 1) {
    uint32_t m = 0;
    for (uint32_t t = k; t; t >>= 1) ++m;
    len += m;
    k = m - 1;
  }
  return len;
}

// msgs / tables / bytes as the decode entry points receive them. packed: tables[k] points to the
// four info words of message k and bytes[k] says how much of the message buffer may be read;
// otherwise tables[k] is the offset table and bytes (optional) bounds the payload.
int resolve_peers(const void* const* msgs, const uint64_t* const* tables, const uint64_t* bytes, bool packed,
                  uint32_t K, uint64_t n, uint32_t bucket, uint32_t s, int code_kind, PeerSet* ps) {
  if (!msgs) return QSGD_ERR_NULL;
  if (K < 1 || K > QSGD_MAX_PEERS) return QSGD_ERR_PEERS;
  if (code_kind != QSGD_CODE_FIXED && (!tables || (packed && !bytes))) return QSGD_ERR_NULL;
  const FixedLayout L = make_fixed_layout(n, bucket, s);
  ps->packed = (packed && code_kind != QSGD_CODE_FIXED) ? 1u : 0u;
  for (uint32_t k = 0; k < K; ++k) {
    ps->bound[k] = (bytes && code_kind != QSGD_CODE_FIXED) ? bytes[k] : 0ull;
    if (!msgs[k]) return QSGD_ERR_NULL;
    if (!aligned16(msgs[k])) return QSGD_ERR_ALIGN;
    const uint8_t* m = static_cast<const uint8_t*>(msgs[k]);
    if (code_kind == QSGD_CODE_FIXED) {
      ps->A[k] = reinterpret_cast<const float*>(m);
      ps->sign[k] = reinterpret_cast<const uint32_t*>(m + L.off_sign);
      ps->level[k] = reinterpret_cast<const uint32_t*>(m + L.off_level);
      ps->payload[k] = nullptr; ps->table[k] = nullptr;
    } else {
      if (!tables[k]) return QSGD_ERR_NULL;
      if (reinterpret_cast<uintptr_t>(tables[k]) & 7u) return QSGD_ERR_ALIGN;
      ps->A[k] = nullptr; ps->sign[k] = nullptr; ps->level[k] = nullptr;
      ps->payload[k] = reinterpret_cast<const uint32_t*>(m);
      ps->table[k] = tables[k];
    }
  }
  return QSGD_OK;
}

}  // namespace
}  // namespace qsgd

using namespace qsgd;

extern "C" {

size_t qsgd_message_capacity(uint64_t n, uint32_t bucket, uint32_t s, int code_kind) {
  if (check_shape(n, bucket, s, code_kind) != QSGD_OK) return 0;
  if (code_kind == QSGD_CODE_FIXED) return (size_t)make_fixed_layout(n, bucket, s).total;
  const uint64_t B = (n + bucket - 1) / bucket;
  // longest string: every coordinate nonzero at the level with the longest code, every gap 1
  const uint64_t per = code_kind == QSGD_CODE_ELIAS ? 2ull + host_elias_len(s) : 1ull + host_elias_len(s + 1);
  const uint64_t bits = 32ull * B + n * per;
  return (size_t)(align16((bits + 7) / 8) + 8 * (B + 1));
}

size_t qsgd_workspace_bytes(uint64_t n, uint32_t bucket, uint32_t s, int code_kind) {
  if (check_shape(n, bucket, s, code_kind) != QSGD_OK) return 0;
  if (code_kind == QSGD_CODE_FIXED) return 0;
  return elias_workspace_bytes(n, bucket, s);
}

int qsgd_fixed_layout(uint64_t n, uint32_t bucket, uint32_t s, uint64_t* layout) {
  if (!layout) return QSGD_ERR_NULL;
  const int st = check_shape(n, bucket, s, QSGD_CODE_FIXED);
  if (st) return st;
  const FixedLayout L = make_fixed_layout(n, bucket, s);
  layout[0] = L.off_sign; layout[1] = L.off_level; layout[2] = L.total; layout[3] = L.lb;
  return QSGD_OK;
}

int qsgd_encode(const float* g, uint64_t n, uint32_t bucket, uint32_t s, int norm_kind,
                int code_kind, uint64_t seed, uint32_t step, uint32_t worker, void* out,
                size_t out_capacity, uint64_t* out_bits, void* workspace, uint32_t* status_dev,
                qsgd_stream_t stream) {
  if (!g || !out || !out_bits || !status_dev) return QSGD_ERR_NULL;
  int st = check_shape(n, bucket, s, code_kind);
  if (st) return st;
  if (norm_kind != QSGD_NORM_L2 && norm_kind != QSGD_NORM_MAX) return QSGD_ERR_KIND;
  if (!aligned16(g) || !aligned16(out)) return QSGD_ERR_ALIGN;
  cudaStream_t cs = static_cast<cudaStream_t>(stream);
  if (code_kind == QSGD_CODE_FIXED) {
    const FixedLayout L = make_fixed_layout(n, bucket, s);
    if (out_capacity < L.total) return QSGD_ERR_CAPACITY;
    return launch_quantize_fixed(g, n, bucket, s, norm_kind, seed, step, worker,
                                 static_cast<uint8_t*>(out), status_dev, out_bits, nullptr, no_map(), cs);
  }
  if (!workspace) return QSGD_ERR_NULL;
  if (!aligned16(workspace)) return QSGD_ERR_ALIGN;
  const uint64_t B = (n + bucket - 1) / bucket;
  if (out_capacity < align16(4 * B) + 8 * (B + 1)) return QSGD_ERR_CAPACITY;   // scales + table
  return launch_elias_encode(g, n, bucket, s, norm_kind, code_kind == QSGD_CODE_ELIAS_DENSE, seed,
                             step, worker, static_cast<uint8_t*>(out), out_capacity, out_bits,
                             static_cast<uint8_t*>(workspace), status_dev, no_map(), cs);
}

static int decode_any(const void* const* msgs, const uint64_t* const* tables, const uint64_t* bytes, bool packed,
                      uint32_t K, uint64_t n, uint32_t bucket, uint32_t s, int code_kind, float* out, bool fused,
                      float eta, uint32_t* status_dev, qsgd_stream_t stream) {
  if (!out || !status_dev) return QSGD_ERR_NULL;
  int st = check_shape(n, bucket, s, code_kind);
  if (st) return st;
  if (!aligned16(out)) return QSGD_ERR_ALIGN;
  PeerSet ps;
  st = resolve_peers(msgs, tables, bytes, packed, K, n, bucket, s, code_kind, &ps);
  if (st) return st;
  cudaStream_t cs = static_cast<cudaStream_t>(stream);
  if (code_kind == QSGD_CODE_FIXED) return launch_decode_fixed(ps, K, n, bucket, s, out, fused, eta, no_map(), cs);
  return launch_decode_elias(ps, K, n, bucket, s, code_kind == QSGD_CODE_ELIAS_DENSE, out, fused, eta,
                             status_dev, no_map(), cs);
}

int qsgd_decode_accumulate(const void* const* msgs, const uint64_t* const* tables, const uint64_t* payload_bytes,
                           uint32_t K, uint64_t n, uint32_t bucket, uint32_t s, int code_kind, float* acc,
                           uint32_t* status_dev, qsgd_stream_t stream) {
  return decode_any(msgs, tables, payload_bytes, false, K, n, bucket, s, code_kind, acc, false, 0.f, status_dev, stream);
}

int qsgd_decode_accumulate_packed(const void* const* msgs, const uint64_t* const* infos, const uint64_t* msg_bytes,
                                  uint32_t K, uint64_t n, uint32_t bucket, uint32_t s, int code_kind, float* acc,
                                  uint32_t* status_dev, qsgd_stream_t stream) {
  return decode_any(msgs, infos, msg_bytes, true, K, n, bucket, s, code_kind, acc, false, 0.f, status_dev, stream);
}

int qsgd_decode_sgd_step_packed(const void* const* msgs, const uint64_t* const* infos, const uint64_t* msg_bytes,
                                uint32_t K, uint64_t n, uint32_t bucket, uint32_t s, int code_kind, float* x,
                                float eta, uint32_t* status_dev, qsgd_stream_t stream) {
  return decode_any(msgs, infos, msg_bytes, true, K, n, bucket, s, code_kind, x, true, eta, status_dev, stream);
}

int qsgd_sgd_step(float* x, const float* acc, float eta, uint32_t K, uint64_t n,
                  qsgd_stream_t stream) {
  if (!x || !acc) return QSGD_ERR_NULL;
  if (n == 0) return QSGD_ERR_SIZE;
  if (K < 1 || K > QSGD_MAX_PEERS) return QSGD_ERR_PEERS;
  if (!aligned16(x) || !aligned16(acc)) return QSGD_ERR_ALIGN;
  return launch_sgd_step(x, acc, eta, K, n, static_cast<cudaStream_t>(stream));
}

int qsgd_decode_sgd_step(const void* const* msgs, const uint64_t* const* tables, const uint64_t* payload_bytes,
                         uint32_t K, uint64_t n, uint32_t bucket, uint32_t s, int code_kind, float* x,
                         float eta, uint32_t* status_dev, qsgd_stream_t stream) {
  return decode_any(msgs, tables, payload_bytes, false, K, n, bucket, s, code_kind, x, true, eta, status_dev, stream);
}

// ---- per-tensor policy --------------------------------------------------------------------------
int qsgd_policy_plan_sizes(const uint64_t* tensor_sizes, uint32_t T, uint32_t bucket, uint64_t min_quantized,
                           uint64_t* n_buckets, uint64_t* n_raw_segments, uint64_t* n_raw) {
  if (!tensor_sizes || !n_buckets || !n_raw_segments || !n_raw) return QSGD_ERR_NULL;
  if (bucket < 32 || bucket > QSGD_MAX_BUCKET || (bucket & 31u)) return QSGD_ERR_BUCKET;
  uint64_t nb = 0, ns = 0, nr = 0, total = 0;
  for (uint32_t t = 0; t < T; ++t) {
    const uint64_t m = tensor_sizes[t];
    total += m;
    if (m >= min_quantized && m > 0) nb += (m + bucket - 1) / bucket;
    else if (m > 0) { ++ns; nr += m; }
  }
  if (total == 0) return QSGD_ERR_SIZE;
  *n_buckets = nb; *n_raw_segments = ns; *n_raw = nr;
  return QSGD_OK;
}

int qsgd_policy_plan(const uint64_t* tensor_sizes, uint32_t T, uint32_t bucket, uint64_t min_quantized,
                     uint64_t* bucket_src, uint32_t* bucket_len, uint64_t* raw_src, uint64_t* raw_start,
                     uint32_t* quads) {
  uint64_t nb, ns, nr;
  const int st = qsgd_policy_plan_sizes(tensor_sizes, T, bucket, min_quantized, &nb, &ns, &nr);
  if (st) return st;
  if (!quads || (nb && (!bucket_src || !bucket_len)) || !raw_start || (ns && !raw_src)) return QSGD_ERR_NULL;
  uint64_t off = 0, b = 0, seg = 0, r = 0;
  bool q = true;
  for (uint32_t t = 0; t < T; ++t) {
    const uint64_t m = tensor_sizes[t];
    if (m >= min_quantized && m > 0) {
      for (uint64_t c = 0; c < m; c += bucket, ++b) {
        bucket_src[b] = off + c;
        bucket_len[b] = (uint32_t)(m - c < bucket ? m - c : bucket);
        q = q && ((bucket_src[b] | bucket_len[b]) & 3ull) == 0;
      }
    } else if (m > 0) {
      raw_src[seg] = off;
      raw_start[seg] = r;
      ++seg;
      r += m;
    }
    off += m;
  }
  raw_start[seg] = r;
  *quads = q ? 1u : 0u;
  return QSGD_OK;
}

static int check_policy(const qsgd_policy* plan, uint32_t bucket, uint32_t s, int code_kind) {
  if (!plan) return QSGD_ERR_NULL;
  if (plan->n == 0 || (plan->n_buckets == 0 && plan->n_raw == 0)) return QSGD_ERR_SIZE;
  if (plan->n_buckets && (!plan->bucket_src || !plan->bucket_len)) return QSGD_ERR_NULL;
  if (plan->n_raw && (!plan->raw_src || !plan->raw_start || plan->n_raw_segments == 0)) return QSGD_ERR_NULL;
  return check_shape(plan->n_buckets ? plan->n_buckets * bucket : 1, bucket, s, code_kind);
}

static RawSegments raw_of(const qsgd_policy* plan) {
  return RawSegments{plan->raw_src, plan->raw_start, plan->n_raw_segments, plan->n_raw};
}

static BucketMap map_of(const qsgd_policy* plan) {
  return BucketMap{plan->bucket_src, plan->bucket_len, plan->quads};
}

size_t qsgd_policy_message_capacity(const qsgd_policy* plan, uint32_t bucket, uint32_t s, int code_kind) {
  if (check_policy(plan, bucket, s, code_kind) != QSGD_OK) return 0;
  const size_t prefix = (size_t)align16(4 * plan->n_raw);
  return prefix + (plan->n_buckets ? qsgd_message_capacity(plan->n_buckets * bucket, bucket, s, code_kind) : 0);
}

size_t qsgd_policy_workspace_bytes(const qsgd_policy* plan, uint32_t bucket, uint32_t s, int code_kind) {
  if (check_policy(plan, bucket, s, code_kind) != QSGD_OK || plan->n_buckets == 0) return 0;
  return qsgd_workspace_bytes(plan->n_buckets * bucket, bucket, s, code_kind);
}

int qsgd_policy_encode(const float* g, const qsgd_policy* plan, uint32_t bucket, uint32_t s, int norm_kind,
                       int code_kind, uint64_t seed, uint32_t step, uint32_t worker, void* out,
                       size_t out_capacity, uint64_t* out_bits, void* workspace, uint32_t* status_dev,
                       qsgd_stream_t stream) {
  if (!g || !out || !out_bits || !status_dev) return QSGD_ERR_NULL;
  int st = check_policy(plan, bucket, s, code_kind);
  if (st) return st;
  if (norm_kind != QSGD_NORM_L2 && norm_kind != QSGD_NORM_MAX) return QSGD_ERR_KIND;
  if (!aligned16(g) || !aligned16(out)) return QSGD_ERR_ALIGN;
  const size_t prefix = (size_t)align16(4 * plan->n_raw);
  if (out_capacity < prefix) return QSGD_ERR_CAPACITY;
  cudaStream_t cs = static_cast<cudaStream_t>(stream);
  const uint64_t nc = plan->n_buckets * bucket;
  if (nc) {
    uint8_t* body = static_cast<uint8_t*>(out) + prefix;
    const size_t cap = out_capacity - prefix;
    if (code_kind == QSGD_CODE_FIXED) {
      if (cap < make_fixed_layout(nc, bucket, s).total) return QSGD_ERR_CAPACITY;
      st = launch_quantize_fixed(g, nc, bucket, s, norm_kind, seed, step, worker, body, status_dev, out_bits,
                                 nullptr, map_of(plan), cs);
    } else {
      if (!workspace) return QSGD_ERR_NULL;
      if (!aligned16(workspace)) return QSGD_ERR_ALIGN;
      if (cap < align16(4 * plan->n_buckets) + 8 * (plan->n_buckets + 1)) return QSGD_ERR_CAPACITY;
      st = launch_elias_encode(g, nc, bucket, s, norm_kind, code_kind == QSGD_CODE_ELIAS_DENSE, seed, step,
                               worker, body, cap, out_bits, static_cast<uint8_t*>(workspace), status_dev,
                               map_of(plan), cs);
    }
    if (st) return st;
  }
  return launch_raw_gather(g, raw_of(plan), static_cast<float*>(out), out_bits, nc != 0, cs);
}

static int policy_decode(const void* const* msgs, const uint64_t* const* tables, const uint64_t* payload_bytes,
                         uint32_t K, const qsgd_policy* plan, uint32_t bucket, uint32_t s, int code_kind, float* out,
                         bool fused, float eta, uint32_t* status_dev, qsgd_stream_t stream) {
  if (!out || !status_dev || !msgs) return QSGD_ERR_NULL;
  int st = check_policy(plan, bucket, s, code_kind);
  if (st) return st;
  if (K < 1 || K > QSGD_MAX_PEERS) return QSGD_ERR_PEERS;
  if (!aligned16(out)) return QSGD_ERR_ALIGN;
  const size_t prefix = (size_t)align16(4 * plan->n_raw);
  const void* body[QSGD_MAX_PEERS];
  const float* raw[QSGD_MAX_PEERS];
  for (uint32_t k = 0; k < K; ++k) {
    if (!msgs[k]) return QSGD_ERR_NULL;
    if (!aligned16(msgs[k])) return QSGD_ERR_ALIGN;
    body[k] = static_cast<const uint8_t*>(msgs[k]) + prefix;
    raw[k] = static_cast<const float*>(msgs[k]);
  }
  cudaStream_t cs = static_cast<cudaStream_t>(stream);
  const uint64_t nc = plan->n_buckets * bucket;
  if (nc) {
    PeerSet ps;
    st = resolve_peers(body, tables, payload_bytes, false, K, nc, bucket, s, code_kind, &ps);
    if (st) return st;
    if (code_kind == QSGD_CODE_FIXED) st = launch_decode_fixed(ps, K, nc, bucket, s, out, fused, eta, map_of(plan), cs);
    else st = launch_decode_elias(ps, K, nc, bucket, s, code_kind == QSGD_CODE_ELIAS_DENSE, out, fused, eta,
                                  status_dev, map_of(plan), cs);
    if (st) return st;
  }
  return launch_raw_decode(raw, K, raw_of(plan), out, fused, eta, cs);
}

int qsgd_policy_decode_accumulate(const void* const* msgs, const uint64_t* const* tables, const uint64_t* payload_bytes,
                                  uint32_t K, const qsgd_policy* plan, uint32_t bucket, uint32_t s, int code_kind,
                                  float* acc, uint32_t* status_dev, qsgd_stream_t stream) {
  return policy_decode(msgs, tables, payload_bytes, K, plan, bucket, s, code_kind, acc, false, 0.f, status_dev, stream);
}

int qsgd_policy_decode_sgd_step(const void* const* msgs, const uint64_t* const* tables, const uint64_t* payload_bytes,
                                uint32_t K, const qsgd_policy* plan, uint32_t bucket, uint32_t s, int code_kind,
                                float* x, float eta, uint32_t* status_dev, qsgd_stream_t stream) {
  return policy_decode(msgs, tables, payload_bytes, K, plan, bucket, s, code_kind, x, true, eta, status_dev, stream);
}

const char* qsgd_status_string(int status) {
  switch (status) {
    case QSGD_OK: return "ok";
    case QSGD_ERR_NULL: return "a required pointer is null";
    case QSGD_ERR_SIZE: return "n must lie in [1, 2^32]";
    case QSGD_ERR_BUCKET: return "bucket must be a multiple of 32 in [32, 4096]";
    case QSGD_ERR_LEVELS: return "s must lie in [1, 255]";
    case QSGD_ERR_ALIGN: return "pointer not 16-byte aligned";
    case QSGD_ERR_CAPACITY: return "output capacity too small";
    case QSGD_ERR_PEERS: return "K must lie in [1, 64]";
    case QSGD_ERR_KIND: return "unknown norm or code kind";
    case QSGD_ERR_NO_DEVICE: return "no usable CUDA device";
    case QSGD_ERR_SCRATCH: return "problem too large for the built-in scratch array";
    default: return status > 0 ? cudaGetErrorString((cudaError_t)status) : "unknown status";
  }
}

int qsgd_set_launch_chaining(int on) { return set_launch_chaining(on != 0) ? 1 : 0; }

void qsgd_test_set_wait_polls(uint32_t polls) { set_quantize_poll_limit(polls); }

uint32_t qsgd_test_default_wait_polls(void) { return default_quantize_poll_limit(); }

uint64_t qsgd_launch_count(void) { return g_launches.load(std::memory_order_relaxed); }

void qsgd_profile_enable(int on) { g_profile.store(on ? 1 : 0, std::memory_order_relaxed); }

int qsgd_profile_kernel_count(void) { return (int)kKernCount; }

const char* qsgd_profile_kernel_name(int id) {
  return (id >= 0 && id < (int)kKernCount) ? kKernelNames[id] : "";
}

int qsgd_profile_collect(double* total_ms, uint64_t* launches) {
  std::vector<TimedLaunch> mine;
  {
    std::lock_guard<std::mutex> lk(g_prof_mu);
    mine.swap(g_timed);
  }
  for (int i = 0; i < (int)kKernCount; ++i) { total_ms[i] = 0.0; launches[i] = 0; }
  int rc = 0;
  for (const TimedLaunch& t : mine) {
    float ms = 0.f;
    cudaError_t e = cudaEventSynchronize(t.b);
    if (e == cudaSuccess) e = cudaEventElapsedTime(&ms, t.a, t.b);
    if (e != cudaSuccess) rc = (int)e;
    else { total_ms[t.id] += (double)ms; launches[t.id] += 1; }
    cudaEventDestroy(t.a);
    cudaEventDestroy(t.b);
  }
  return rc;
}

}  // extern "C"
