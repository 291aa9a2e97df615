/*
 * FastSGD oracle -- TEST INFRASTRUCTURE, NOT THE PRODUCT.
 *
 * A plain, slow, single-threaded CPU statement of what the FastSGD gradient
 * encoder / decoder computes (Sec. 3.1-3.3, Eq. 2-4, Algorithms 1 and 2 of the
 * paper), written to be checked against the paper by eye.  It shares no code,
 * header, table or constant generator with the CUDA library; only tests, the
 * smoke check and the CPU-baseline leg of the benchmark may call it.
 *
 * Every function below is pinned by the CPU test-suite against facts that do
 * not come from this file (the paper's worked examples, exact rational
 * arithmetic, brute force, a second parser).  The only statements of the paper
 * that stay "parity unpinned" are its data-dependent measurements (bits per
 * key on KDD12, the message-size ratios): the dataset is not available.
 *
 * Build: gcc -O2 -ffp-contract=off -fno-fast-math -std=c99 -shared -fPIC
 */
#ifndef FASTSGD_ORACLE_H
#define FASTSGD_ORACLE_H

#include <stdint.h>
#include <stddef.h>

#ifdef __cplusplus
extern "C" {
#endif

/* Hyper-parameters of the method: base b (Eq. 3), threshold tau (Sec. 3.2,
 * Phase 3), length-flag size l (Sec. 3.3, Phase 5) and the container's group
 * size T = 2^group_log2 (one independent Algorithm-2 instance per T indices). */
typedef struct {
    double   base;
    uint32_t tau;
    uint32_t flag_bits;
    uint32_t group_log2;
    uint32_t reserved;
} fsgo_params;

/* status words that can appear in a stream header */
enum {
    FSGO_OK            = 0,
    FSGO_ERR_NONFINITE = 1,   /* sum of |v| is not finite                     */
    FSGO_ERR_CAPACITY  = 2,   /* output buffer too small for the stream       */
    FSGO_ERR_TIMEOUT   = 3    /* never produced by the oracle                 */
};
/* status words a decoder reports */
enum {
    FSGO_DEC_BAD_MAGIC      = 16,
    FSGO_DEC_BAD_VERSION    = 17,
    FSGO_DEC_BAD_STATUS     = 18,
    FSGO_DEC_N_MISMATCH     = 19,
    FSGO_DEC_PARAM_MISMATCH = 20,
    FSGO_DEC_TRUNCATED      = 21,
    FSGO_DEC_BAD_DIRECTORY  = 22,
    FSGO_DEC_BAD_KEY        = 23,
    FSGO_DEC_BAD_CODE       = 24   /* code byte with L > tau */
};
#define FSGO_BAD_PARAM (-3)

/* ---- the steps, one function each ------------------------------------ */

/* sum = sum_i |v_i| (Algorithm 1, first step; numerator of Eq. 2), evaluated
 * in fp64 on the balanced binary tree over index ranges aligned to powers of
 * two: node(lo,1) = |v[lo]| (0 beyond n), node(lo,len) = node(lo,len/2) +
 * node(lo+len/2,len/2). */
double fsgo_abs_sum(const float *v, uint64_t n);

/* P[k] = b^k by P[0]=1, P[k]=P[k-1]*b, and the quantisation boundaries
 * B[k] = sum / P[k], k = 0..tau.  B[tau] is the early-stop threshold tau_e of
 * Algorithm 1.  Returns 0, or FSGO_BAD_PARAM if b<=1, tau not in 1..128 or
 * b^tau overflows. */
int fsgo_tables(double sum, double base, uint32_t tau, double *P, double *B);

/* L = ceil(log_b(sum/|v|)) (Eq. 2 and Eq. 3) evaluated as the least k in
 * [0,tau] with |v| >= B[k]; returns tau+1 when there is none (the value is
 * filtered out).  `a` is |v| widened to fp64. */
uint32_t fsgo_quantise(double a, const double *B, uint32_t tau);

/* Algorithm 1 as a whole: keys (indices) and signed codes q = +-L of the kept
 * values in index order, and the sum.  L = 0 is raised to 1.  keys/codes need
 * room for n entries.  Returns 0 / FSGO_BAD_PARAM / FSGO_ERR_NONFINITE. */
int fsgo_value_encode(const float *v, uint64_t n, double base, uint32_t tau,
                      uint64_t *keys, int32_t *codes, uint64_t *d, double *sum);

/* one-byte form of a signed code: bit 7 = sign, bits 0..6 = L-1 */
uint8_t fsgo_code_byte(int32_t q);
int32_t fsgo_code_from_byte(uint8_t c);

/* number of bits of x (0 for x = 0) */
uint32_t fsgo_bitlen(uint64_t x);
/* M = max(1, bitlen(maxDelta)); widths[f] = ceil((f+1)*M / 2^l), f < 2^l */
void fsgo_widths(uint32_t M, uint32_t l, uint32_t *widths);
/* smallest flag f whose width holds delta */
uint32_t fsgo_length_flag(uint64_t delta, const uint32_t *widths, uint32_t l);

/* Algorithm 2 exactly as printed: one delta chain from preKey = 0, one M, and
 * BK = flag||delta for each key in turn.  Writes the sequence as '0'/'1'
 * characters (NUL-terminated) into `bk` (capacity `cap` characters) and the
 * value of M into *M_out.  Returns the number of bits, or -1 if cap is too
 * small.  Used for pins only. */
int64_t fsgo_key_encode_paper(const uint64_t *keys, uint64_t d, uint32_t l,
                              char *bk, uint64_t cap, uint32_t *M_out);

/* ---- the container ---------------------------------------------------- */

uint64_t fsgo_compress_bound(uint64_t n, const fsgo_params *p);

/* encoder: gradient -> stream.  *total = bytes produced.  Returns the status
 * that was written to the header (or FSGO_BAD_PARAM, nothing written). */
int fsgo_compress(const float *v, uint64_t n, const fsgo_params *p,
                  uint8_t *out, uint64_t cap, uint64_t *total);

/* container writer for already chosen (key, signed code) pairs; keys strictly
 * increasing and < n.  Used by fsgo_compress and by the key-codec pins. */
int fsgo_write_stream(const uint64_t *keys, const int32_t *codes, uint64_t d,
                      uint64_t n, double sum, const fsgo_params *p,
                      uint8_t *out, uint64_t cap, uint64_t *total);

/* decoder phases 1-2 (+ code bytes): keys and signed codes of a stream.
 * keys/codes need room for header d entries.  Returns FSGO_OK or a decoder
 * status. */
int fsgo_parse(const uint8_t *stream, uint64_t bytes, uint64_t n,
               const fsgo_params *p, uint64_t *keys, int32_t *codes,
               uint64_t *d, double *sum);

/* decoder phases 1-4 and the aggregation: dense[k] += sign * (float)B[L]. */
int fsgo_decompress_accumulate(const uint8_t *stream, uint64_t bytes,
                               uint64_t n, const fsgo_params *p, float *dense);

/* The encoder on a gradient given as `count` key-value pairs (strictly ascending
 * keys < n): by definition the stream of the dense vector that holds values[j]
 * at keys[j] and zeros elsewhere.  FSGO_BAD_PARAM if the keys do not ascend or
 * reach n. */
int fsgo_compress_kv(const uint64_t *keys, const float *values, uint64_t count,
                     uint64_t n, const fsgo_params *p, uint8_t *out, uint64_t cap,
                     uint64_t *total);

/* Model update on the decoded coordinates only (Adam as printed in the
 * experimental set-up: m = beta1 m + (1 - beta1) g, v = beta2 v + (1 - beta2) g^2,
 * theta = theta - lr / sqrt(v + eps) * m, no bias correction).  g is the sum, in
 * the order given, of the decoded streams; a coordinate whose g is zero (in no
 * stream, or cancelled) keeps theta, m and v.  Every operation is one IEEE
 * single-precision operation, in the order written in the source.  Returns the
 * first stream's error, if any, with nothing updated. */
typedef struct { float lr, beta1, beta2, eps; } fsgo_adam;
int fsgo_sparse_adam_update(const uint8_t *const *streams, const uint64_t *bytes,
                            uint32_t num_streams, uint64_t n, const fsgo_params *p,
                            const fsgo_adam *h, float *theta, float *m, float *v);

#ifdef __cplusplus
}
#endif
#endif
