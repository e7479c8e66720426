/*
 * qsgd.h -- C ABI of the QSGD gradient codec for NVIDIA B200 (sm_100a).
 *
 * The library implements the data-parallel hot path of QSGD (Alistarh et al., arXiv
 * 1610.02132): Encode = stochastic quantizer Q_s (Section 3.1, Eq. 2; bucketing and max-norm
 * scaling of Section 4) followed by a lossless code -- either fixed-width bit fields (the
 * "2/4/8-bit QSGD" of Section 5) or the Elias-coded string S of Section 3.1 / Appendix A.2 --
 * and Decode of K peers' messages summed into the step of Algorithm 1,
 * x <- x - (eta / K) * sum_k Decode(M^k).
 *
 * Conventions
 *   - Every pointer is a DEVICE pointer owned by the caller unless its comment says "host".
 *     The library allocates no device memory and never synchronises the host: each call
 *     validates its arguments, enqueues kernels on `stream` and returns.
 *   - Return value: 0 = launched; < 0 = invalid argument (nothing was launched), see
 *     QSGD_ERR_*; > 0 = a cudaError_t reported by a launch.
 *   - Faults found by kernels (message capacity exceeded, malformed Elias stream) are OR-ed
 *     into status_dev[0] (QSGD_DEV_*). The caller zeroes that word and reads it back when it
 *     synchronises. A kernel that finds a fault skips the offending write; it never traps.
 *   - Messages carry no header: n, bucket, s and the code kind are call arguments on both
 *     sides, as in the paper where sender and receiver agree on s and n.
 *   - All fp32 arithmetic is round-to-nearest-even without FMA contraction, in the order
 *     stated below, so a message and a decoded update are bit-reproducible.
 *   - Inputs must be finite with s * max|g| representable in fp32; otherwise values are
 *     unspecified but all memory accesses stay in bounds.
 *
 * Notation: n coordinates; bucket size d; B = ceil(n / d) buckets, the last one possibly
 * shorter, each with its own scale; s quantization levels; lb = 1, 2, 4, 8 level bits for
 * s <= 1, 3, 15, 255.
 *
 * Fixed-width message (QSGD_CODE_FIXED): three regions, each zero-padded to a multiple of 16
 * bytes: fp32 scale A[B] | sign bitmap, coordinate i at bit (i % 32) of u32 word i / 32, set
 * when the value is negative and its level is nonzero | level fields, coordinate i at bits
 * [(i * lb) % 32, +lb) of u32 word (i * lb) / 32.
 *
 * Elias message (QSGD_CODE_ELIAS): the per-bucket strings S of Section 3.1 (32 bits of the
 * IEEE-754 pattern of A, then for every nonzero level, in index order: Elias(distance to the
 * previous nonzero; for the first one its 1-based position), one sign bit, Elias(level))
 * concatenated without padding. Stream bit t is bit 31 - (t % 32) of u32 word t / 32. The
 * payload is zero-padded to a multiple of 16 bytes and followed by a table of B + 1 u64 bit
 * offsets (offset of each bucket's string; last entry = payload bits). The table is an
 * addition of this format (the paper codes one vector and needs none); sizes are reported
 * with and without it. QSGD_CODE_ELIAS_DENSE is the variant Code'_s of Appendix A.3: after
 * the 32 bits of A, every coordinate sends one sign bit and Elias(level + 1).
 */
#ifndef QSGD_H_
#define QSGD_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

#define QSGD_NORM_L2 0  /* A = ||v||_2 of the bucket (Eq. 2)              */
#define QSGD_NORM_MAX 1 /* A = max |v_i| of the bucket (Section 4)        */

#define QSGD_CODE_FIXED 0
#define QSGD_CODE_ELIAS 1
#define QSGD_CODE_ELIAS_DENSE 2

#define QSGD_MAX_COORDS (1ull << 32) /* largest n accepted (16 GiB of fp32 gradient per call) */
#define QSGD_MAX_BUCKET 4096
#define QSGD_MAX_LEVELS 255
#define QSGD_MAX_PEERS 64

#define QSGD_OK 0
#define QSGD_ERR_NULL (-1)      /* a required pointer is null                         */
#define QSGD_ERR_SIZE (-2)      /* n == 0 or n > QSGD_MAX_COORDS                      */
#define QSGD_ERR_BUCKET (-3)    /* bucket not a multiple of 32 in [32, 4096]          */
#define QSGD_ERR_LEVELS (-4)    /* s outside [1, 255]                                 */
#define QSGD_ERR_ALIGN (-5)     /* a pointer is not 16-byte aligned                   */
#define QSGD_ERR_CAPACITY (-6)  /* out_capacity below the minimum for this call       */
#define QSGD_ERR_PEERS (-7)     /* K outside [1, 64]                                  */
#define QSGD_ERR_KIND (-8)      /* unknown norm_kind or code_kind                     */
#define QSGD_ERR_NO_DEVICE (-9) /* no usable CUDA device / kernel image for this GPU  */
#define QSGD_ERR_SCRATCH (-10)  /* problem too large for the library's built-in scratch */

/* Size of the scratch array built into the library for qsgd_encode_elias_static. */
#define QSGD_STATIC_SCRATCH_BYTES (32u << 20)

#define QSGD_DEV_CAPACITY 1u  /* encoded message would exceed out_capacity             */
#define QSGD_DEV_OVERRUN 2u   /* an Elias code runs past the end of its bucket string  */
#define QSGD_DEV_POSITION 4u  /* a decoded position lies outside its bucket            */
#define QSGD_DEV_LEVEL 8u     /* a decoded level lies outside [1, s]                   */
#define QSGD_DEV_TABLE 16u    /* offset table not ascending / bucket shorter than 32   */
#define QSGD_DEV_TIMEOUT 32u  /* a bounded wait inside a kernel gave up                */

typedef void* qsgd_stream_t; /* a cudaStream_t; NULL is the default stream */

/* Worst-case bytes of one message (Section 3.1 string lengths; fixed-width: exact size). */
size_t qsgd_message_capacity(uint64_t n, uint32_t bucket, uint32_t s, int code_kind);

/* Bytes of scratch qsgd_encode needs for the Elias kinds (0 for QSGD_CODE_FIXED). */
size_t qsgd_workspace_bytes(uint64_t n, uint32_t bucket, uint32_t s, int code_kind);

/* Fixed-width layout: layout[0] = byte offset of the sign bitmap, [1] = byte offset of the
 * level fields, [2] = total bytes, [3] = level bits lb. `layout` is a host pointer. */
int qsgd_fixed_layout(uint64_t n, uint32_t bucket, uint32_t s, uint64_t* layout);

/*
 * Encode (Algorithm 1, "M^i <- Encode(g^i)"; Section 3.1, Eq. 2 and the string S).
 * Per bucket: scale A in fp32, the exact maximum or the 2-norm. The 2-norm is the correctly
 * rounded square root of a sum of squares that the streaming kernels (power-of-two bucket, at
 * least 4096 coordinates) accumulate in fp32 -- a chain of 16 fused multiply-adds per thread,
 * then a shuffle tree over the bucket's lanes, then, for buckets of 1024 and more, up to 8
 * sequential adds across warps -- and redo in fp64 when that sum leaves [8e-28, 1e30] (a sum of
 * exactly zero included: squares below 1.4e-45 vanish in fp32 although the norm is representable);
 * the generic kernel (other shapes, ragged tail) sums 8 squares in fp32 and those partial sums in
 * fp64, and redoes a bucket in fp64 likewise. Either way A lies within 1e-6 relative of the exact norm (at most 29 roundings of 2^-24
 * on the sum, halved by the root), but the two kernels may give last-place differences for the
 * same bucket, so a message is reproducible for a given (n, bucket), not across shapes. A scale
 * below the smallest normal fp32 makes a zero bucket (A = +0, all levels 0). Per coordinate i (global index): u = Philox4x32-10(counter = (i / 4 lo,
 * i / 4 hi, step, worker), key = seed lo, hi) word i % 4, top 24 bits times 2^-24;
 * level = min(floor((s * |g_i|) * (1 / A) + u), s).
 *   g            n fp32 values, 16-byte aligned, read once
 *   out          message buffer of out_capacity bytes, 16-byte aligned, fully overwritten
 *                up to the message length
 *   out_bits     4 u64 words written on the stream: [0] payload bits (fixed-width: 8 * bytes),
 *                [1] byte offset of the offset table in `out` (0 for fixed), [2] message
 *                bytes, [3] 0
 *   workspace    qsgd_workspace_bytes() of scratch, 16-byte aligned (may be NULL for fixed)
 *   status_dev   one u32, OR-ed with QSGD_DEV_CAPACITY when out_capacity is too small
 */
int qsgd_encode(const float* g, uint64_t n, uint32_t bucket, uint32_t s, int norm_kind,
                int code_kind, uint64_t seed, uint32_t step, uint32_t worker, void* out,
                size_t out_capacity, uint64_t* out_bits, void* workspace, uint32_t* status_dev,
                qsgd_stream_t stream);

/*
 * Decode K messages and sum them (Algorithm 1, "g^l <- Decode(M^l)" and the sum):
 * acc_i = ((+0 + g^0_i) + g^1_i) + ... in ascending k, where g^k_i = +-(A * (level / s)).
 *   msgs    host array of K device pointers to messages (16-byte aligned)
 *   tables  host array of K device pointers to the offset tables (Elias kinds; msgs[k] +
 *           out_bits[1]); NULL for fixed-width. With the table directly behind the payload the
 *           library reads the payload sizes off the pointers and chooses between its decoders on
 *           the host; with tables kept elsewhere it decides on the device (two launches, one of
 *           which returns at once). Results are the same either way.
 *   payload_bytes  host array of K payload lengths in bytes (the padded payload, = out_bits[1]
 *           of each message), or NULL. The decoders read no payload bit at or beyond
 *           8 * payload_bytes[k]: a table whose last entry claims more is refused with
 *           QSGD_DEV_TABLE before any payload read. With NULL the bound is the table's own address
 *           when the table lies behind the payload (as Encode writes it); for a table kept
 *           elsewhere there is then no bound and the caller vouches for the table. In every case a
 *           payload must be readable for 16 bytes past its padded length (true when its table
 *           follows it): the bit window prefetches two words ahead.
 *   acc     n fp32 values, overwritten
 */
int qsgd_decode_accumulate(const void* const* msgs, const uint64_t* const* tables,
                           const uint64_t* payload_bytes, uint32_t K, uint64_t n, uint32_t bucket,
                           uint32_t s, int code_kind, float* acc, uint32_t* status_dev,
                           qsgd_stream_t stream);

/* SGD step (Algorithm 1, last line): c = eta / K once; x_i <- x_i - c * acc_i. */
int qsgd_sgd_step(float* x, const float* acc, float eta, uint32_t K, uint64_t n,
                  qsgd_stream_t stream);

/* Decode, sum and step in one pass over x; bit-identical to the two calls above. */
int qsgd_decode_sgd_step(const void* const* msgs, const uint64_t* const* tables,
                         const uint64_t* payload_bytes, uint32_t K, uint64_t n, uint32_t bucket,
                         uint32_t s, int code_kind, float* x, float eta, uint32_t* status_dev,
                         qsgd_stream_t stream);

/*
 * The same two calls for messages exactly as Encode left them (Algorithm 1, "receive M^l, decode"):
 * a packaging that needs no host read-back between Encode and Decode. Where the offset table of an
 * Elias message starts is known only on the device (out_bits[1], written by Encode on the stream);
 * instead of table pointers the caller passes
 *   infos      host array of K DEVICE pointers to the four out_bits words of each message (8-byte
 *              aligned; for a received message: wherever its info words were put), and
 *   msg_bytes  host array of K byte counts: how much of message buffer k may be read (its capacity
 *              as allocated is fine).
 * The kernels take table k at msgs[k] + infos[k][1]; that place must be 16-byte aligned with all
 * 8 * (B + 1) table bytes inside msg_bytes[k], and infos[k][1] bounds the payload, else
 * QSGD_DEV_TABLE is raised and nothing of that message is read. The choice among the Elias
 * decoders is made on the device (two launches, one returns at once). For QSGD_CODE_FIXED infos
 * and msg_bytes are ignored (may be NULL). Results are bit-identical to the calls above.
 */
int qsgd_decode_accumulate_packed(const void* const* msgs, const uint64_t* const* infos,
                                  const uint64_t* msg_bytes, uint32_t K, uint64_t n, uint32_t bucket,
                                  uint32_t s, int code_kind, float* acc, uint32_t* status_dev,
                                  qsgd_stream_t stream);
int qsgd_decode_sgd_step_packed(const void* const* msgs, const uint64_t* const* infos,
                                const uint64_t* msg_bytes, uint32_t K, uint64_t n, uint32_t bucket,
                                uint32_t s, int code_kind, float* x, float eta, uint32_t* status_dev,
                                qsgd_stream_t stream);

/* Text for a negative return code ("ok" for 0). Host pointer to a static string. */
const char* qsgd_status_string(int status);

/* Number of kernels this library has launched in this process (all calls, all streams). */
uint64_t qsgd_launch_count(void);

/*
 * Launch chaining (the paper has no counterpart). By default every kernel of the library is launched
 * with programmatic stream serialization: its launch is prepared while the kernel ahead of it in the
 * stream still runs, and the kernel itself waits for that kernel to complete before it touches global
 * memory, so the stream's order of reads and writes is the ordinary one. qsgd_set_launch_chaining(0)
 * makes later launches of this process plain stream-ordered launches (for a profiler or a debugger
 * that wants kernels strictly one after the other); nonzero turns chaining back on. Returns the
 * previous setting.
 */
int qsgd_set_launch_chaining(int on);

/*
 * TEST HOOK, not part of the codec (the paper has no counterpart). The streaming encoder waits for
 * its bulk copies with bounded polling; when a wait runs out the warp (or CTA) raises
 * QSGD_DEV_TIMEOUT in status_dev, stops encoding, still waits -- with the full built-in bound --
 * for the copies it has in flight, and returns. qsgd_test_set_wait_polls sets the bound of the
 * main-loop waits for later launches of this process (0 = every such wait gives up at once), so a
 * test can drive that path without any fault; qsgd_test_default_wait_polls returns the built-in
 * bound to restore. Output written by a launch that timed out is unspecified inside the message
 * buffer and never outside it.
 */
void qsgd_test_set_wait_polls(uint32_t polls);
uint32_t qsgd_test_default_wait_polls(void);

/*
 * Elias Encode that allocates nothing and needs no caller-supplied workspace. (The paper has no
 * counterpart: this is a packaging of qsgd_encode for one kind of caller.)
 *
 * Who needs it: code that may not obtain device memory at the moment it has to encode -- a
 * gradient hook that fires inside a framework whose caching allocator is locked or whose memory
 * budget was fixed at start-up, a communication plug-in that is handed buffers but no allocator,
 * a latency-critical thread that must not enter cudaMalloc (which can synchronise the whole
 * device). Such a caller still passes the gradient, the message buffer, the four info words and
 * the status word, as for qsgd_encode; what it cannot provide is the qsgd_workspace_bytes() of
 * scratch. Here that scratch is one array of QSGD_STATIC_SCRATCH_BYTES (32 MiB) compiled into
 * the library as a device global, so every GPU that loads the library carries it until the
 * process exits. The call itself performs no cudaMalloc, cudaFree or other allocating call.
 *
 *   - code_kind must be QSGD_CODE_ELIAS or QSGD_CODE_ELIAS_DENSE (fixed-width needs no scratch:
 *     use qsgd_encode). Results are bit-identical to qsgd_encode with the same arguments.
 *   - Limit: qsgd_workspace_bytes(n, bucket, s, code_kind) must not exceed
 *     qsgd_static_scratch_bytes(); e.g. bucket 512, s = 15 fits up to about 47 million
 *     coordinates. Larger problems are rejected with QSGD_ERR_SCRATCH and nothing is launched.
 *   - The first call on each device looks up the device address of the built-in array (a host
 *     side query, done with that device current and cached per device). Make that first call
 *     outside of any stream capture.
 *   - All calls on one device share the one array, which keeps whatever the previous call left
 *     in it; every region the kernels read is rewritten by the same call first, so nothing needs
 *     clearing between calls. Two calls that overlap on the GPU (different streams, or several
 *     host threads) race on the array and corrupt each other's messages: serialise them.
 */
size_t qsgd_static_scratch_bytes(void);
int qsgd_encode_elias_static(const float* g, uint64_t n, uint32_t bucket, uint32_t s, int norm_kind,
                             int code_kind, uint64_t seed, uint32_t step, uint32_t worker, void* out,
                             size_t out_capacity, uint64_t* out_bits, uint32_t* status_dev,
                             qsgd_stream_t stream);

/*
 * Per-tensor policy (Section 5, "Protocol": tensors with fewer than 10K elements are not
 * quantized, and buckets are cut so that they fit the tensors).
 *
 * The flat gradient g[n] is the concatenation of T tensors. A tensor with fewer than
 * `min_quantized` elements is "raw": its fp32 values travel unchanged. Every other tensor is cut
 * into buckets of `bucket` elements that start at the tensor's first element; the last bucket of a
 * tensor may be shorter. The quantized tensors form a "compact" vector in which each tensor is
 * padded with zeros to whole buckets (zeros change no norm and quantize to level 0); Encode and
 * Decode of the compact vector are exactly qsgd_encode / qsgd_decode_* on n_buckets * bucket
 * coordinates, the uniform of a coordinate being keyed by its compact index. The padding exists
 * in no buffer: the kernels read and write each bucket at its own place in g / x.
 *
 * Policy message = raw values in tensor order (fp32, zero-padded to 16 bytes) followed by the
 * ordinary message of the compact vector. out_bits: [0] 32 * n_raw plus the ordinary [0],
 * [1] byte offset of the offset table inside `out` (0 for QSGD_CODE_FIXED), [2] message bytes,
 * [3] bytes of the raw region in front.
 *
 * qsgd_policy_plan_sizes / qsgd_policy_plan run on the host and touch no GPU. The first returns
 * the array lengths, the second fills caller-owned HOST arrays:
 *   bucket_src[n_buckets], bucket_len[n_buckets]   place in g and length of every bucket,
 *   raw_src[n_raw_segments], raw_start[n_raw_segments + 1]   place in g of every raw tensor and
 *                                                   its offset in the raw region (last = n_raw),
 * and returns in *quads whether every bucket place and length is a multiple of 4 elements (then
 * the kernels may use 16-byte accesses and bulk copies; otherwise they fall back to narrower ones).
 * The caller copies the arrays to the device and hands them over in a qsgd_policy. Returns
 * QSGD_OK, QSGD_ERR_NULL, QSGD_ERR_BUCKET or QSGD_ERR_SIZE (no elements at all).
 */
typedef struct {
  const uint64_t* bucket_src;  /* device */
  const uint32_t* bucket_len;  /* device */
  uint64_t n_buckets;
  const uint64_t* raw_src;     /* device */
  const uint64_t* raw_start;   /* device */
  uint64_t n_raw_segments;
  uint64_t n_raw;
  uint64_t n;                  /* elements of the flat gradient */
  uint32_t quads;              /* as returned by qsgd_policy_plan */
} qsgd_policy;

int qsgd_policy_plan_sizes(const uint64_t* tensor_sizes, uint32_t T, uint32_t bucket, uint64_t min_quantized,
                           uint64_t* n_buckets, uint64_t* n_raw_segments, uint64_t* n_raw);
int qsgd_policy_plan(const uint64_t* tensor_sizes, uint32_t T, uint32_t bucket, uint64_t min_quantized,
                     uint64_t* bucket_src, uint32_t* bucket_len, uint64_t* raw_src, uint64_t* raw_start,
                     uint32_t* quads);

/* Worst-case bytes of one policy message, and scratch bytes of qsgd_policy_encode. */
size_t qsgd_policy_message_capacity(const qsgd_policy* plan, uint32_t bucket, uint32_t s, int code_kind);
size_t qsgd_policy_workspace_bytes(const qsgd_policy* plan, uint32_t bucket, uint32_t s, int code_kind);

/*
 * Encode / Decode under the policy. Arguments as for qsgd_encode, qsgd_decode_accumulate and
 * qsgd_decode_sgd_step, with the plan in place of n; `plan` is a host pointer to a struct of device
 * pointers. msgs[k] points to the start of policy message k (its raw region), tables[k] to its
 * offset table (msgs[k] + out_bits[1]), payload_bytes[k] (optional, as for qsgd_decode_accumulate) is
 * the padded payload length out_bits[1] - out_bits[3]. acc (n floats) is overwritten at every coordinate; x is
 * updated at every coordinate; fused and unfused results are equal bit for bit. Errors as for the
 * ordinary calls. Launches: the ordinary encode or decode kernels plus one small kernel for the
 * raw tensors.
 */
int qsgd_policy_encode(const float* g, const qsgd_policy* plan, uint32_t bucket, uint32_t s, int norm_kind,
                       int code_kind, uint64_t seed, uint32_t step, uint32_t worker, void* out,
                       size_t out_capacity, uint64_t* out_bits, void* workspace, uint32_t* status_dev,
                       qsgd_stream_t stream);
int qsgd_policy_decode_accumulate(const void* const* msgs, const uint64_t* const* tables,
                                  const uint64_t* payload_bytes, uint32_t K, const qsgd_policy* plan,
                                  uint32_t bucket, uint32_t s, int code_kind, float* acc,
                                  uint32_t* status_dev, qsgd_stream_t stream);
int qsgd_policy_decode_sgd_step(const void* const* msgs, const uint64_t* const* tables,
                                const uint64_t* payload_bytes, uint32_t K, const qsgd_policy* plan,
                                uint32_t bucket, uint32_t s, int code_kind, float* x, float eta,
                                uint32_t* status_dev, qsgd_stream_t stream);

/*
 * Per-kernel timing (measurement aid; the paper has no counterpart). While enabled, every
 * kernel launch of the library is bracketed by two CUDA events on its stream.
 * qsgd_profile_collect waits for the recorded events, adds each kernel's elapsed time and
 * launch count into the host arrays total_ms[] / launches[] (qsgd_profile_kernel_count()
 * entries, indexed by kernel id) and forgets them. Returns 0 or a cudaError_t.
 */
void qsgd_profile_enable(int on);
int qsgd_profile_kernel_count(void);
const char* qsgd_profile_kernel_name(int id);
int qsgd_profile_collect(double* total_ms, uint64_t* launches);

#ifdef __cplusplus
}
#endif
#endif /* QSGD_H_ */
