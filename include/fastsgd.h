/*
 * fastsgd.h -- C ABI of the B200 (sm_100a) FastSGD gradient codec.
 *
 * The calls follow the paper's statement of the problem (arxiv 2112.04291):
 * a worker's gradient, read as key-value pairs (Sec. 2.2), goes through the
 * gradient value encoder (Sec. 3.2, Eq. 2-3, Algorithm 1: reciprocal mapper,
 * logarithm quantisation, threshold filter) and the gradient key encoder
 * (Sec. 3.3, Eq. 4, Algorithm 2: delta keys, length flags, bit-level binary
 * encoding); the decoder (Sec. 3.1, decoder phases 1-4) inverts both and the
 * decoded gradients of the W workers are aggregated (Sec. 2.1).
 *
 * Conventions
 *   - "device" pointers are CUDA global-memory addresses on the current
 *     device, "host" pointers are ordinary process memory.
 *   - The caller owns every buffer.  The library allocates nothing; its scratch
 *     memory is the workspace the caller registers with fastsgd_set_workspace.
 *   - fastsgd_compress and fastsgd_decompress_accumulate only enqueue kernels
 *     on `stream` (a cudaStream_t passed as void*) and return at once.  The
 *     library keeps one workspace per device (the one registered while that
 *     device was current); all calls on a device must be issued on one stream
 *     (or otherwise serialised): they share that workspace.  Different devices
 *     of one process are independent of each other.
 *   - Return value: 0 or a negative FASTSGD_E_* for what the host can see.
 *     What only the device can see is reported in a status word: the stream
 *     header's for compress (fastsgd_stream_info), the workspace's for
 *     decompress (fastsgd_decode_status).
 *   - There is no CPU fallback.
 *
 * Stream layout (little-endian; the paper fixes only that the codes travel
 * with `sum` and the keys as the binary sequence BK):
 *   header, 64 bytes: u32 magic "FSG1", u32 version, u32 status, u32 tau,
 *     u64 n, u64 d, u64 total_bytes, f64 sum, f64 b, u8 l, u8 group_log2,
 *     u16 0, u32 G
 *   directory, G = ceil(n / 2^group_log2) entries: u32 count | M << 24,
 *     u32 offset of the group's blob in 4-byte words from the stream start
 *   blobs, in group order: count code bytes (bit 7 sign, bits 0-6 L-1), count
 *     length flags of l bits, the deltas in the widths the flags select,
 *     zero bits up to a multiple of 32; all fields most significant bit first.
 *   Each group is one instance of Algorithm 2 over the kept keys that fall
 *   in [g*T, (g+1)*T), T = 2^group_log2, with preKey starting at g*T.
 *   When status != 0 only the header is defined (d = 0, total_bytes = 64).
 */
#ifndef FASTSGD_H
#define FASTSGD_H

#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

/* Hyper-parameters (Sec. 4.2 recommends b ~ 1.1, tau = 128, l = 2). */
typedef struct fastsgd_params {
    double   base;        /* b > 1, with b^tau finite (Eq. 3)                        */
    uint32_t tau;         /* threshold, 1..128: kept codes L satisfy 1 <= L <= tau    */
    uint32_t flag_bits;   /* l, 1..5: size of the length flag (Sec. 3.3, Phase 5)     */
    uint32_t group_log2;  /* log2 of the group size T, 8..20 (see fastsgd_compress); 14 is the fast path */
    uint32_t reserved;    /* must be 0                                               */
} fastsgd_params;

/* host-visible errors (return values) */
#define FASTSGD_OK                 0
#define FASTSGD_E_NULL            (-1)
#define FASTSGD_E_ALIGN           (-2)   /* grad / out / stream_in not 16-byte aligned, dense_out not 4-byte */
#define FASTSGD_E_BAD_PARAM       (-3)
#define FASTSGD_E_BAD_N           (-4)   /* n = 0 or n >= 2^31                                                */
#define FASTSGD_E_CAPACITY        (-5)   /* out_bytes smaller than header + directory                        */
#define FASTSGD_E_NO_WORKSPACE    (-6)   /* no workspace registered, or too small for this n                 */
#define FASTSGD_E_NOT_IMPLEMENTED (-7)   /* valid parameters this build has no kernel for                    */
#define FASTSGD_E_CUDA            (-8)   /* a CUDA runtime call failed                                       */
#define FASTSGD_E_TRUNCATED       (-9)   /* decompress: fewer than 64 bytes given                            */
#define FASTSGD_E_TOO_LARGE       (-10)  /* fastsgd_abs_sum_noalloc: n above FASTSGD_NOALLOC_MAX_N           */

/* device-visible status words */
#define FASTSGD_ST_OK              0
#define FASTSGD_ST_NONFINITE       1     /* compress: sum of |v| is Inf or NaN                               */
#define FASTSGD_ST_CAPACITY        2     /* compress: stream does not fit in out_bytes                       */
#define FASTSGD_ST_TIMEOUT         3     /* a bounded wait between thread blocks ran out (see fastsgd_compress) */
#define FASTSGD_ST_BAD_MAGIC      16
#define FASTSGD_ST_BAD_VERSION    17
#define FASTSGD_ST_BAD_STATUS     18     /* decompress: the stream's own status is not OK                    */
#define FASTSGD_ST_N_MISMATCH     19
#define FASTSGD_ST_PARAM_MISMATCH 20
#define FASTSGD_ST_TRUNCATED      21
#define FASTSGD_ST_BAD_DIRECTORY  22
#define FASTSGD_ST_BAD_KEY        23     /* a decoded key leaves its group or repeats                        */
#define FASTSGD_ST_BAD_CODE       24     /* a code byte with L > tau                                         */

/*
 * Encoder (Sec. 3.2 Algorithm 1 followed by Sec. 3.3 Algorithm 2).
 *   grad       device, n floats, 16-byte aligned; read twice, never written
 *   n          number of gradient entries D_m, 1 <= n < 2^31
 *   params     host
 *   out        device, 16-byte aligned, receives the stream
 *   out_bytes  capacity of `out` in bytes (by value); at least
 *              64 + 8*G; fastsgd_compress_bound(n, params) always suffices.
 *              The produced length is header.total_bytes (device memory;
 *              fastsgd_stream_info reads it back).
 *   stream     cudaStream_t
 * Computes sum = sum|v_i| on a fixed fp64 pairwise tree, the boundaries
 * B_k = sum / b^k, keeps entry i iff |v_i| >= B_tau (the early-stop threshold
 * tau_e), gives it the code L = min{k : |v_i| >= B_k} = ceil(log_b(sum/|v_i|))
 * (raised to 1 if 0) with the sign of v_i, and writes the stream.
 * If the stream does not fit, or the sum is not finite, only a 64-byte header
 * carrying the status is written.  Nothing outside out[0, out_bytes) is
 * written.
 * Group sizes: T = 2^14 is what the fused kernel is built for (its tile is the
 * group).  Any other group_log2 in 8..20 takes a general path: the sum kernel,
 * a kernel that selects the kept entries (i, v_i), |v_i| >= B_tau, into a list
 * in the workspace, and the list encoder of fastsgd_compress_kv on that list
 * (three reads of the gradient, about 1.5 times the fused kernel's time; a list
 * beyond 4.5 M pairs does not fit and the list encoder then walks the dense
 * gradient itself, a warp per group, which is slow for large groups).  The
 * stream is the one the definition gives for that group size (the paper's
 * Algorithm 2 has no groups: it is the case T >= n).  Below 2^8:
 * FASTSGD_E_NOT_IMPLEMENTED.  The decoder takes the same range as long as the
 * stream has at most 2^17 groups.
 * The kernel is launched cooperatively (all its thread blocks resident at
 * once, two per SM) and its blocks wait for one another with bounded waits; if
 * one of them runs out (it should not on a GPU the kernel has to itself) every
 * stream of that launch reports FASTSGD_ST_TIMEOUT, and the workspace must be
 * registered again before the next call: once fastsgd_stream_info or
 * fastsgd_decode_status has returned that status, every compress and
 * decompress call fails with FASTSGD_E_NO_WORKSPACE until
 * fastsgd_set_workspace is called again.
 */
int fastsgd_compress(const float* grad, uint64_t n, const fastsgd_params* params,
                     void* out, uint64_t out_bytes, void* stream);

/*
 * The same encoder for the gradients of several workers (Sec. 2.1: W workers
 * each hold a gradient of the same model), all of length n and compressed with
 * the same parameters, each into its own stream.
 *   grads   host array of num_grads device pointers (each 16-byte aligned)
 *   outs    host array of num_grads device pointers (each 16-byte aligned),
 *           every one with room for out_bytes bytes
 * Every stream is byte for byte what fastsgd_compress produces for that
 * gradient.  Up to 8 gradients share one kernel launch: thread blocks that are
 * done with one gradient start on the next while the others finish.
 */
int fastsgd_compress_batch(const float* const* grads, uint64_t n, const fastsgd_params* params,
                           void* const* outs, uint64_t out_bytes, uint32_t num_grads, void* stream);

/*
 * The encoder for a gradient given as key-value pairs (Sec. 2.2 states the
 * problem on the D non-zero pairs (k_j, v_j) of a D_m-dimensional gradient;
 * the sparse models of Sec. 4 produce it in this form).
 *   keys    device, `count` strictly ascending 32-bit keys, each < n
 *   values  device, the matching fp32 values (zeros allowed: never kept)
 *   n       D_m; out, out_bytes, params, stream as for fastsgd_compress
 * The stream is, byte for byte, the one fastsgd_compress writes for the dense
 * vector that holds values[j] at keys[j] and zeros elsewhere: the sum is
 * formed on the same tree (zeros add exactly nothing), the groups are the
 * same.  Nothing of size n is read, formed or written except the directory
 * (8 bytes per group) and one pass over the per-chunk sums (8 bytes per 2^14
 * indices): cost in proportion to count and to n / 2^14.  Any group_log2 in
 * 1..20.  Keys that do not ascend or reach n give an unspecified stream, never
 * an access outside the buffers.  One cooperative launch (a warp per 32 pairs;
 * two grid barriers with bounded waits, FASTSGD_ST_TIMEOUT as for
 * fastsgd_compress).
 */
int fastsgd_compress_kv(const uint32_t* keys, const float* values, uint64_t count, uint64_t n,
                        const fastsgd_params* params, void* out, uint64_t out_bytes, void* stream);

/*
 * Decoder and aggregation (Sec. 3.1 decoder phases 1-4; Sec. 2.1 aggregation).
 *   stream_in  device, 16-byte aligned, a stream made by fastsgd_compress
 *   bytes      number of valid bytes at stream_in (>= header.total_bytes)
 *   n, params  must equal the header's, else FASTSGD_ST_N_MISMATCH /
 *              FASTSGD_ST_PARAM_MISMATCH
 *   dense_out  device, n floats: dense_out[k] += sign * (float)(sum / b^L) for
 *              every kept (k, L); never cleared, so that the streams of several
 *              workers add up in call order
 * A damaged stream never causes an access outside stream_in[0, bytes) or
 * dense_out[0, n); its status is recorded (fastsgd_decode_status) and the
 * contents of dense_out are then unspecified.  Header-level damage leaves
 * dense_out untouched.
 */
int fastsgd_decompress_accumulate(const void* stream_in, uint64_t bytes, uint64_t n,
                                  const fastsgd_params* params, float* dense_out, void* stream);

/*
 * The same decoder and aggregation for the streams of several workers in one
 * launch (Sec. 2.1: the W workers' decoded gradients are aggregated).
 *   streams_in   host array of num_streams device pointers (each 16-byte
 *                aligned), bytes the matching host array of valid byte counts
 * The result equals that of num_streams calls of
 * fastsgd_decompress_accumulate in the given order, bit for bit: a group's
 * streams are applied one after the other.  Up to 8 streams go into one
 * kernel launch; longer lists take several launches.
 */
int fastsgd_decompress_accumulate_batch(const void* const* streams_in, const uint64_t* bytes,
                                        uint32_t num_streams, uint64_t n, const fastsgd_params* params,
                                        float* dense_out, void* stream);

/*
 * Model update on the decoded coordinates only (Sec. 4.1, "Implementation":
 * the models are trained with Adam; Table of the running-time breakdown, part
 * "model updating").  Hyper-parameters of the two Adam equations of Sec. 4.1.
 */
typedef struct fastsgd_adam {
    float lr;      /* eta */
    float beta1;
    float beta2;
    float eps;
} fastsgd_adam;

/*
 * Decodes the workers' streams and applies one Adam step to the coordinates
 * that received a non-zero aggregated gradient; all other coordinates keep
 * theta, m and v (the update costs time in proportion to the kept entries, not
 * to n).
 *   streams_in, bytes, num_streams, n, params   as for
 *                fastsgd_decompress_accumulate_batch
 *   hyper        host pointer
 *   grad_scratch device, n floats, ALL ZERO on entry and all zero again when
 *                the call has run: the aggregated gradient g lives here between
 *                aggregation and update (the caller clears it once, when it
 *                allocates it)
 *   theta, m, v  device, n floats each, updated in place where g != 0:
 *                  m = beta1 * m + (1 - beta1) * g
 *                  v = beta2 * v + (1 - beta2) * g * g
 *                  theta = theta - lr / sqrt(v + eps) * m
 *                every operation one IEEE fp32 operation (round to nearest, no
 *                fused multiply-add), in the order written
 * g is the sum of the decoded streams in the given order, exactly as
 * fastsgd_decompress_accumulate_batch forms it.  Up to 8 streams: one launch
 * (the warp or block that decodes a group aggregates it and then updates its
 * coordinates); more: two launches per 8 streams, aggregation of all of them,
 * then the update.  Errors and damaged streams as for
 * fastsgd_decompress_accumulate_batch (theta, m, v and grad_scratch are then
 * unspecified, never accessed out of bounds).
 */
int fastsgd_sparse_adam_update_batch(const void* const* streams_in, const uint64_t* bytes,
                                     uint32_t num_streams, uint64_t n, const fastsgd_params* params,
                                     const fastsgd_adam* hyper, float* grad_scratch,
                                     float* theta, float* m, float* v, void* stream);

/*
 * The same update with the model's state kept as one array of four floats per
 * coordinate, (theta, m, v, g): a coordinate's step then reads and writes one
 * 16-byte entry instead of one 32-byte sector in each of three arrays (the
 * update of scattered coordinates is bound by memory transactions, Sec. 4.1's
 * "model updating" part).  g is the scratch of the call above, interleaved.
 *   state        device, 16-byte aligned, 4 n floats: state[4 i + 0] = theta_i,
 *                [4 i + 1] = m_i, [4 i + 2] = v_i, [4 i + 3] = g_i; every g_i
 *                ZERO on entry and zero again when the call has run
 *   other arguments, the arithmetic, the order of the streams, errors and
 *                damaged streams: as for fastsgd_sparse_adam_update_batch
 * One launch.  At most 8 streams and groups of at most 2^14 indices
 * (group_log2 <= 14): otherwise FASTSGD_E_NOT_IMPLEMENTED.
 */
int fastsgd_sparse_adam_update_packed_batch(const void* const* streams_in, const uint64_t* bytes,
                                            uint32_t num_streams, uint64_t n, const fastsgd_params* params,
                                            const fastsgd_adam* hyper, float* state, void* stream);

/*
 * Algorithm 2 exactly as printed (Sec. 3.3): one delta chain over all kept keys
 * starting from preKey = 0, one M = max(1, bitlen(maxDelta)), and the binary
 * sequence BK = flag || delta for each key in turn, most significant bit first
 * (level f of the 2^l levels holds ceil((f+1) M / 2^l) bits; a delta takes the
 * lowest level that holds it).  The product stream of fastsgd_compress uses the
 * same code per group of 2^14 indices; this call states the paper's own format
 * and its size per key (Tables "space cost of gradient key").
 *   keys       device, d ascending 32-bit keys (a first key of 0 gives a delta
 *              of 0; later deltas are >= 1)
 *   flag_bits  l, 1..5
 *   out        device, 16-byte aligned, fastsgd_key_encode_paper_bound(d, l)
 *              bytes at least (else FASTSGD_E_CAPACITY):
 *                u32 M | u32 l | u64 number of bits in BK
 *                u64 index[ceil(d / 2048)]: bit offset in BK of key 2048 i
 *                BK, zero bits up to a multiple of 32
 * Four small launches on `stream`; no workspace.  Keys that do not ascend give
 * an unspecified BK, never an access outside the buffers.
 */
uint64_t fastsgd_key_encode_paper_bound(uint64_t d, uint32_t flag_bits);
int fastsgd_key_encode_paper(const uint32_t* keys, uint64_t d, uint32_t flag_bits,
                             void* out, uint64_t out_bytes, void* stream);

/* ---- helpers, not on the timed path (no counterpart in the paper) ---------- */

/* worst-case stream size in bytes (every entry kept, every delta at the widest
 * level); 0 for invalid arguments */
uint64_t fastsgd_compress_bound(uint64_t n, const fastsgd_params* params);

/* bytes of device scratch the two calls need for gradients of up to n entries */
uint64_t fastsgd_workspace_bytes(uint64_t n, const fastsgd_params* params);

/* Registers caller-owned device memory (256-byte aligned) as the library's
 * scratch and initialises it on `stream`.  The memory must stay valid until
 * another workspace is registered. */
int fastsgd_set_workspace(void* dev_ptr, uint64_t bytes, void* stream);

/* Synchronises `stream`, then copies total_bytes, d and status out of a
 * stream's header (any pointer may be NULL). */
int fastsgd_stream_info(const void* stream_in, void* stream, uint64_t* total_bytes,
                        uint64_t* d, int* status);

/* Synchronises `stream`, returns in *status the status of the decompress calls
 * since the last query (FASTSGD_ST_OK if none failed; else that of the lowest
 * damaged group seen), and clears it. */
int fastsgd_decode_status(void* stream, int* status);

/* Step 1 of Algorithm 1 alone: *sum_out (device, one double) = sum|v_i| on the
 * same fp64 pairwise tree fastsgd_compress uses.  Uses the workspace. */
int fastsgd_abs_sum(const float* grad, uint64_t n, double* sum_out, void* stream);

/*
 * The same sum for callers that cannot hand the library any scratch memory.
 * (The paper has no counterpart: this is a packaging variant of step 1 of
 * Algorithm 1, bit-identical to fastsgd_abs_sum.)
 *
 * Who needs it: code that runs where device memory cannot be obtained at call
 * time -- a plug-in inside a host application that owns the whole device heap,
 * a latency-critical loop that must not hit cudaMalloc's implicit device-wide
 * synchronisation or its failure under memory pressure, a component that is
 * only ever given its input and output buffers.  Such a caller cannot register
 * a workspace either, so the per-tile partial sums and the block counter live
 * in a fixed array inside the library's own device image instead
 * (about 129 KiB, held by every GPU that loads the library until the process
 * exits).  The price is a size limit: n <= FASTSGD_NOALLOC_MAX_N, otherwise
 * FASTSGD_E_TOO_LARGE is returned and nothing is launched.
 *
 *   grad     device, n floats, 16-byte aligned
 *   sum_out  device, one double, 8-byte aligned
 * The call allocates nothing and frees nothing, neither through the CUDA
 * runtime nor through any library.  The first call on a device looks the
 * array's device address up and queries launch limits (once per device, with
 * that device current); make that first call outside any stream capture.
 * All calls on a device share the one array, which keeps what the previous
 * call left: the call clears the part that must start at zero itself, but two
 * calls that overlap on the GPU (different streams, no ordering) race on it --
 * issue them on one stream or order them yourself.
 */
#define FASTSGD_NOALLOC_MAX_N (1ull << 28)
int fastsgd_abs_sum_noalloc(const float* grad, uint64_t n, double* sum_out, void* stream);

/*
 * Host-buffer forms of the two calls, for callers whose gradients live in host
 * memory: copy in, run the device path, copy the result out, all on `stream`,
 * then synchronise.  `dev_scratch` is caller-owned device memory of at least
 * fastsgd_host_scratch_bytes(n, params) bytes (16-byte aligned).
 *   fastsgd_compress_host: grad_host (n floats) -> out_host (capacity
 *     out_bytes); *produced = bytes written to out_host; *status = header status.
 *   fastsgd_decompress_accumulate_host: decodes `num_streams` streams (host
 *     pointers streams_host[i] of bytes[i] bytes each, in that order) into one
 *     dense vector and copies it to dense_host (n floats).  accumulate = 0
 *     starts from zero, accumulate = 1 from dense_host's contents.
 *     *status = decoder status.
 */
uint64_t fastsgd_host_scratch_bytes(uint64_t n, const fastsgd_params* params);
int fastsgd_compress_host(const float* grad_host, uint64_t n, const fastsgd_params* params,
                          void* out_host, uint64_t out_bytes, uint64_t* produced, int* status,
                          void* dev_scratch, uint64_t dev_scratch_bytes, void* stream);
int fastsgd_decompress_accumulate_host(const void* const* streams_host, const uint64_t* bytes,
                                       uint32_t num_streams, uint64_t n, const fastsgd_params* params,
                                       float* dense_host, int accumulate, int* status,
                                       void* dev_scratch, uint64_t dev_scratch_bytes, void* stream);

const char* fastsgd_strerror(int code);
int fastsgd_version(void);

#ifdef __cplusplus
}
#endif
#endif /* FASTSGD_H */
