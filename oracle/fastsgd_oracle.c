/*
 * FastSGD oracle -- TEST INFRASTRUCTURE, NOT THE PRODUCT (see the header).
 *
 * Plain single-threaded C.  No blocking, fusion or reordering beyond what the
 * paper's algorithms and the stream definition below state.
 *
 * Stream definition (little-endian fields; the paper only says that the codes
 * travel "with sum" and that the keys travel as the binary sequence BK):
 *
 *   header, 64 bytes
 *      0  u32  magic 0x31475346 ("FSG1")
 *      4  u32  version (1)
 *      8  u32  status
 *     12  u32  tau
 *     16  u64  n          number of gradient entries (D_m)
 *     24  u64  d          number of kept entries
 *     32  u64  total_bytes
 *     40  f64  sum        (0.0 when status is FSGO_ERR_NONFINITE)
 *     48  f64  b
 *     56  u8   l ; 57 u8 group_log2 ; 58 u16 zero
 *     60  u32  G = ceil(n / T), T = 2^group_log2
 *   directory, G entries of 8 bytes
 *      u32  count | M << 24      (0 for an empty group)
 *      u32  offset of the group's blob from the start of the stream, in
 *           4-byte words
 *   blobs, one per group, in group order, each a bit sequence
 *      count code bytes | count flags of l bits | the deltas, each in the
 *      width its flag selects | zero bits up to a multiple of 32
 *   Bit t of a blob is bit (7 - t%8) of its byte t/8, and every field is
 *   written most significant bit first, so that the paper's strings ('11' for
 *   3, '0011' for flag 00 + delta 3) appear literally.
 *
 * Each group is one instance of Algorithm 2 over the kept keys inside
 * [g*T, (g+1)*T), with preKey starting at g*T and its own M; the flags and
 * the deltas of a group are stored as two planes instead of interleaved.
 * With T >= n this is Algorithm 2 itself up to that re-arrangement.
 *
 * When status != FSGO_OK only the header is defined (d = 0, total_bytes = 64).
 */
#include "fastsgd_oracle.h"

#include <math.h>
#include <stdlib.h>
#include <string.h>

#define FSGO_MAGIC   0x31475346u
#define FSGO_VERSION 1u
#define FSGO_HEADER  64u

/* ------------------------------------------------------------------ sum */

static double tree_sum(const float *v, uint64_t n, uint64_t lo, uint64_t len)
{
    if (lo >= n) return 0.0;
    if (len == 1) return (double)fabsf(v[lo]);
    uint64_t half = len / 2;
    double left  = tree_sum(v, n, lo, half);
    double right = tree_sum(v, n, lo + half, half);
    return left + right;
}

double fsgo_abs_sum(const float *v, uint64_t n)
{
    uint64_t n2 = 1;
    while (n2 < n) n2 *= 2;
    return tree_sum(v, n, 0, n2);
}

/* --------------------------------------------------------------- tables */

int fsgo_tables(double sum, double base, uint32_t tau, double *P, double *B)
{
    if (!(base > 1.0) || !isfinite(base) || tau < 1 || tau > 128) return FSGO_BAD_PARAM;
    P[0] = 1.0;
    for (uint32_t k = 1; k <= tau; ++k) P[k] = P[k - 1] * base;
    if (!isfinite(P[tau])) return FSGO_BAD_PARAM;
    for (uint32_t k = 0; k <= tau; ++k) B[k] = sum / P[k];
    return 0;
}

/* Eq. 3 with Eq. 2 substituted: ceil(log_b(sum/a)) is the least integer k
 * with b^k >= sum/a, that is with a >= sum / b^k = B[k]. */
uint32_t fsgo_quantise(double a, const double *B, uint32_t tau)
{
    for (uint32_t k = 0; k <= tau; ++k)
        if (a >= B[k]) return k;
    return tau + 1;
}

/* ------------------------------------------- gradient value encoder (Sec. 3.2)
 * By the definitions: S is the sum of all magnitudes (numerator of Eq. 2); an
 * entry is kept iff its code L = ceil(log_b(S/|v|)) (Eq. 3 on Eq. 2) does not
 * exceed tau, which is the test |v| >= S / b^tau (the early-stop threshold);
 * the kept code carries the sign of the value. */

int fsgo_value_encode(const float *v, uint64_t n, double base, uint32_t tau,
                      uint64_t *keys, int32_t *codes, uint64_t *d, double *sum)
{
    double P[129], B[129];
    *d = 0;
    const double S = fsgo_abs_sum(v, n);
    *sum = S;
    int rc = fsgo_tables(S, base, tau, P, B);
    if (rc) return rc;
    if (!isfinite(S)) return FSGO_ERR_NONFINITE;
    uint64_t kept = 0;
    for (uint64_t i = 0; i < n; ++i) {
        const double mag = (double)fabsf(v[i]);
        if (!(mag > 0.0)) continue;                  /* zeros (and only zeros) have no reciprocal */
        if (!(mag >= B[tau])) continue;              /* threshold filter: L <= tau iff |v| >= S / b^tau */
        uint32_t L = fsgo_quantise(mag, B, tau);
        if (L < 1) L = 1;                            /* |v| = S: keeps the sign, still an underestimate */
        keys[kept]  = i;
        codes[kept] = (v[i] < 0.0f) ? -(int32_t)L : (int32_t)L;
        ++kept;
    }
    *d = kept;
    return FSGO_OK;
}

uint8_t fsgo_code_byte(int32_t q)
{
    uint32_t L = (uint32_t)(q < 0 ? -q : q);
    return (uint8_t)(((q < 0) ? 0x80u : 0u) | ((L - 1u) & 0x7Fu));
}

int32_t fsgo_code_from_byte(uint8_t c)
{
    int32_t L = (int32_t)(c & 0x7Fu) + 1;
    return (c & 0x80u) ? -L : L;
}

/* ---------------------------------------------------------- Algorithm 2 */

uint32_t fsgo_bitlen(uint64_t x)
{
    uint32_t b = 0;
    while (x) { ++b; x >>= 1; }
    return b;
}

void fsgo_widths(uint32_t M, uint32_t l, uint32_t *widths)
{
    uint32_t levels = 1u << l;
    for (uint32_t f = 0; f < levels; ++f)
        widths[f] = ((f + 1u) * M + levels - 1u) / levels;   /* ceil((f+1) M / 2^l) */
}

uint32_t fsgo_length_flag(uint64_t delta, const uint32_t *widths, uint32_t l)
{
    uint32_t need = fsgo_bitlen(delta);
    uint32_t levels = 1u << l;
    for (uint32_t f = 0; f < levels; ++f)
        if (need <= widths[f]) return f;
    return levels - 1u;   /* not reached: widths[levels-1] = M >= need */
}

static int64_t put_chars(char *bk, uint64_t cap, int64_t pos, uint64_t value, uint32_t nbits)
{
    if ((uint64_t)pos + nbits + 1 > cap) return -1;
    for (uint32_t i = 0; i < nbits; ++i)
        bk[pos + i] = ((value >> (nbits - 1 - i)) & 1u) ? '1' : '0';
    return pos + nbits;
}

/* Sec. 3.3 by its definitions: the delta keys are the adjacent differences of
 * the ascending keys with the first taken from 0 (Eq. 4); M is the bit length of
 * the largest of them; BK is, key after key, the length flag followed by the
 * delta in the width that flag selects. */
int64_t fsgo_key_encode_paper(const uint64_t *keys, uint64_t d, uint32_t l,
                              char *bk, uint64_t cap, uint32_t *M_out)
{
    uint64_t *delta = (uint64_t *)malloc((d ? d : 1) * sizeof(uint64_t));
    for (uint64_t j = 0; j < d; ++j) delta[j] = keys[j] - (j ? keys[j - 1] : 0u);
    uint64_t widest = 0;
    for (uint64_t j = 0; j < d; ++j) if (delta[j] > widest) widest = delta[j];
    uint32_t M = fsgo_bitlen(widest);
    if (M < 1) M = 1;
    *M_out = M;
    uint32_t widths[32];
    fsgo_widths(M, l, widths);
    int64_t pos = 0;
    for (uint64_t j = 0; j < d && pos >= 0; ++j) {
        const uint32_t flag = fsgo_length_flag(delta[j], widths, l);
        pos = put_chars(bk, cap, pos, flag, l);
        if (pos >= 0) pos = put_chars(bk, cap, pos, delta[j], widths[flag]);
    }
    free(delta);
    if (pos < 0 || (uint64_t)pos + 1 > cap) return -1;
    bk[pos] = '\0';
    return pos;
}

/* ------------------------------------------------------------ container */

static int params_ok(const fsgo_params *p)
{
    if (!p) return 0;
    if (!(p->base > 1.0) || !isfinite(p->base)) return 0;
    if (p->tau < 1 || p->tau > 128) return 0;
    if (p->flag_bits < 1 || p->flag_bits > 5) return 0;
    if (p->group_log2 < 1 || p->group_log2 > 20) return 0;
    if (p->reserved != 0) return 0;
    double P = 1.0;
    for (uint32_t k = 1; k <= p->tau; ++k) P = P * p->base;
    return isfinite(P);
}

static void put_u32(uint8_t *p, uint32_t x) { for (int i = 0; i < 4; ++i) p[i] = (uint8_t)(x >> (8 * i)); }
static void put_u64(uint8_t *p, uint64_t x) { for (int i = 0; i < 8; ++i) p[i] = (uint8_t)(x >> (8 * i)); }
static uint32_t get_u32(const uint8_t *p) { uint32_t x = 0; for (int i = 0; i < 4; ++i) x |= (uint32_t)p[i] << (8 * i); return x; }
static uint64_t get_u64(const uint8_t *p) { uint64_t x = 0; for (int i = 0; i < 8; ++i) x |= (uint64_t)p[i] << (8 * i); return x; }
static void put_f64(uint8_t *p, double x) { uint64_t u; memcpy(&u, &x, 8); put_u64(p, u); }
static double get_f64(const uint8_t *p) { uint64_t u = get_u64(p); double x; memcpy(&x, &u, 8); return x; }

static void write_header(uint8_t *out, uint32_t status, uint64_t n, uint64_t d, uint64_t total,
                         double sum, const fsgo_params *p, uint32_t G)
{
    memset(out, 0, FSGO_HEADER);
    put_u32(out + 0, FSGO_MAGIC);
    put_u32(out + 4, FSGO_VERSION);
    put_u32(out + 8, status);
    put_u32(out + 12, p->tau);
    put_u64(out + 16, n);
    put_u64(out + 24, d);
    put_u64(out + 32, total);
    put_f64(out + 40, sum);
    put_f64(out + 48, p->base);
    out[56] = (uint8_t)p->flag_bits;
    out[57] = (uint8_t)p->group_log2;
    put_u32(out + 60, G);
}

/* set bits [pos, pos+nbits) of a zeroed byte array, most significant first */
static void put_bits(uint8_t *blob, uint64_t pos, uint64_t value, uint32_t nbits)
{
    for (uint32_t i = 0; i < nbits; ++i) {
        uint64_t t = pos + i;
        if ((value >> (nbits - 1 - i)) & 1u)
            blob[t / 8] |= (uint8_t)(1u << (7 - t % 8));
    }
}

static uint64_t get_bits(const uint8_t *blob, uint64_t pos, uint32_t nbits)
{
    uint64_t value = 0;
    for (uint32_t i = 0; i < nbits; ++i) {
        uint64_t t = pos + i;
        value = (value << 1) | ((blob[t / 8] >> (7 - t % 8)) & 1u);
    }
    return value;
}

uint64_t fsgo_compress_bound(uint64_t n, const fsgo_params *p)
{
    if (!params_ok(p) || n == 0) return 0;
    uint64_t T = 1ull << p->group_log2;
    uint64_t G = (n + T - 1) / T;
    /* every entry kept, every delta at the widest level M = group_log2 */
    uint64_t bits_per_key = 8 + p->flag_bits + p->group_log2;
    uint64_t per_group_bytes = ((T * bits_per_key + 31) / 32) * 4;
    return FSGO_HEADER + 8 * G + G * per_group_bytes;
}

int fsgo_write_stream(const uint64_t *keys, const int32_t *codes, uint64_t d,
                      uint64_t n, double sum, const fsgo_params *p,
                      uint8_t *out, uint64_t cap, uint64_t *total)
{
    *total = 0;
    if (!params_ok(p) || n == 0) return FSGO_BAD_PARAM;
    uint32_t l = p->flag_bits;
    uint64_t T = 1ull << p->group_log2;
    uint64_t G64 = (n + T - 1) / T;
    uint32_t G = (uint32_t)G64;
    uint64_t fixed = FSGO_HEADER + 8 * G64;
    if (cap < FSGO_HEADER) return FSGO_BAD_PARAM;

    /* first find the size, then write: a stream that does not fit is not
     * written at all */
    uint64_t need = fixed;
    {
        uint64_t j = 0;
        for (uint64_t g = 0; g < G64; ++g) {
            uint64_t hi = (g + 1) * T, preKey = g * T, maxDelta = 0, j0 = j;
            while (j < d && keys[j] < hi) {
                uint64_t delta = keys[j] - preKey; preKey = keys[j];
                if (maxDelta < delta) maxDelta = delta;
                ++j;
            }
            uint64_t count = j - j0;
            if (count == 0) continue;
            uint32_t M = fsgo_bitlen(maxDelta); if (M < 1) M = 1;
            uint32_t widths[32]; fsgo_widths(M, l, widths);
            uint64_t bits = 8 * count + (uint64_t)l * count;
            preKey = g * T;
            for (uint64_t i = j0; i < j; ++i) {
                uint64_t delta = keys[i] - preKey; preKey = keys[i];
                bits += widths[fsgo_length_flag(delta, widths, l)];
            }
            need += ((bits + 31) / 32) * 4;
        }
    }
    if (need > cap) {
        write_header(out, FSGO_ERR_CAPACITY, n, 0, FSGO_HEADER, sum, p, G);
        *total = FSGO_HEADER;
        return FSGO_ERR_CAPACITY;
    }

    uint8_t *dir = out + FSGO_HEADER;
    uint64_t off_words = fixed / 4;
    uint64_t j = 0;
    for (uint64_t g = 0; g < G64; ++g) {
        /* ---- Algorithm 2 on the keys of this group ---- */
        uint64_t hi = (g + 1) * T, preKey = g * T, maxDelta = 0, j0 = j;
        while (j < d && keys[j] < hi) {
            uint64_t delta = keys[j] - preKey; preKey = keys[j];
            if (maxDelta < delta) maxDelta = delta;
            ++j;
        }
        uint64_t count = j - j0;
        if (count == 0) {
            put_u32(dir + 8 * g, 0);
            put_u32(dir + 8 * g + 4, (uint32_t)off_words);
            continue;
        }
        uint32_t M = fsgo_bitlen(maxDelta); if (M < 1) M = 1;
        uint32_t widths[32]; fsgo_widths(M, l, widths);

        uint8_t *blob = out + 4 * off_words;
        uint64_t code_pos = 0, flag_pos = 8 * count, delta_pos = flag_pos + (uint64_t)l * count;
        uint64_t bits = delta_pos;
        preKey = g * T;
        for (uint64_t i = j0; i < j; ++i) {
            uint64_t delta = keys[i] - preKey; preKey = keys[i];
            bits += widths[fsgo_length_flag(delta, widths, l)];
        }
        uint64_t words = (bits + 31) / 32;
        memset(blob, 0, 4 * words);
        preKey = g * T;
        for (uint64_t i = j0; i < j; ++i) {
            uint64_t delta = keys[i] - preKey; preKey = keys[i];
            uint32_t flag = fsgo_length_flag(delta, widths, l);
            put_bits(blob, code_pos, fsgo_code_byte(codes[i]), 8);   code_pos += 8;
            put_bits(blob, flag_pos, flag, l);                       flag_pos += l;
            put_bits(blob, delta_pos, delta, widths[flag]);          delta_pos += widths[flag];
        }
        put_u32(dir + 8 * g, (uint32_t)count | (M << 24));
        put_u32(dir + 8 * g + 4, (uint32_t)off_words);
        off_words += words;
    }
    write_header(out, FSGO_OK, n, d, 4 * off_words, sum, p, G);
    *total = 4 * off_words;
    return FSGO_OK;
}

int fsgo_compress(const float *v, uint64_t n, const fsgo_params *p,
                  uint8_t *out, uint64_t cap, uint64_t *total)
{
    *total = 0;
    if (!params_ok(p) || n == 0 || cap < FSGO_HEADER) return FSGO_BAD_PARAM;
    uint64_t T = 1ull << p->group_log2;
    uint32_t G = (uint32_t)((n + T - 1) / T);
    uint64_t *keys = (uint64_t *)malloc(n * sizeof(uint64_t));
    int32_t *codes = (int32_t *)malloc(n * sizeof(int32_t));
    uint64_t d = 0; double sum = 0.0;
    int rc = fsgo_value_encode(v, n, p->base, p->tau, keys, codes, &d, &sum);   /* Algorithm 1 */
    if (rc == FSGO_ERR_NONFINITE) {
        write_header(out, FSGO_ERR_NONFINITE, n, 0, FSGO_HEADER, 0.0, p, G);
        *total = FSGO_HEADER;
    } else if (rc == FSGO_OK) {
        rc = fsgo_write_stream(keys, codes, d, n, sum, p, out, cap, total);     /* Algorithm 2 per group */
    }
    free(keys); free(codes);
    return rc;
}

/* ---------------------------------------------------------------- decode */

typedef int (*pair_sink)(void *ctx, uint64_t key, uint8_t code_byte);

static int walk_stream(const uint8_t *s, uint64_t bytes, uint64_t n, const fsgo_params *p,
                       uint64_t *d_out, double *sum_out, pair_sink sink, void *ctx)
{
    if (!params_ok(p) || n == 0) return FSGO_BAD_PARAM;
    if (bytes < FSGO_HEADER) return FSGO_DEC_TRUNCATED;
    if (get_u32(s + 0) != FSGO_MAGIC) return FSGO_DEC_BAD_MAGIC;
    if (get_u32(s + 4) != FSGO_VERSION) return FSGO_DEC_BAD_VERSION;
    if (get_u32(s + 8) != FSGO_OK) return FSGO_DEC_BAD_STATUS;
    if (get_u64(s + 16) != n) return FSGO_DEC_N_MISMATCH;
    uint64_t T = 1ull << p->group_log2;
    uint64_t G = (n + T - 1) / T;
    {
        uint64_t hb = get_u64(s + 48), pb; memcpy(&pb, &p->base, 8);
        if (hb != pb || get_u32(s + 12) != p->tau || s[56] != p->flag_bits ||
            s[57] != p->group_log2 || get_u32(s + 60) != (uint32_t)G)
            return FSGO_DEC_PARAM_MISMATCH;
    }
    uint64_t total = get_u64(s + 32);
    uint64_t fixed = FSGO_HEADER + 8 * G;
    if (total > bytes || total < fixed || total % 4 != 0) return FSGO_DEC_TRUNCATED;
    if (d_out) *d_out = get_u64(s + 24);
    if (sum_out) *sum_out = get_f64(s + 40);

    uint32_t l = p->flag_bits;
    const uint8_t *dir = s + FSGO_HEADER;
    uint64_t expect_off = fixed / 4;
    for (uint64_t g = 0; g < G; ++g) {
        uint32_t a = get_u32(dir + 8 * g);
        uint64_t off = get_u32(dir + 8 * g + 4);
        uint64_t count = a & 0xFFFFFFu;
        uint32_t M = a >> 24;
        uint64_t lo = g * T, hi = (g + 1) * T < n ? (g + 1) * T : n;
        uint64_t next_off = (g + 1 < G) ? get_u32(dir + 8 * (g + 1) + 4) : total / 4;
        if (off != expect_off || next_off < off || next_off > total / 4) return FSGO_DEC_BAD_DIRECTORY;
        if (count == 0) {
            if (a != 0 || next_off != off) return FSGO_DEC_BAD_DIRECTORY;
            continue;
        }
        if (count > hi - lo || M < 1 || M > p->group_log2) return FSGO_DEC_BAD_DIRECTORY;
        uint32_t widths[32]; fsgo_widths(M, l, widths);
        const uint8_t *blob = s + 4 * off;
        uint64_t avail_bits = 32 * (next_off - off);
        uint64_t flag_pos = 8 * count, delta_pos = flag_pos + (uint64_t)l * count;
        if (delta_pos > avail_bits) return FSGO_DEC_BAD_DIRECTORY;
        /* phase 1: the flags give every delta's width, hence the blob's length */
        uint64_t bits = delta_pos;
        for (uint64_t i = 0; i < count; ++i)
            bits += widths[get_bits(blob, flag_pos + (uint64_t)l * i, l)];
        if ((bits + 31) / 32 != next_off - off) return FSGO_DEC_BAD_DIRECTORY;
        /* phase 2: running sum of the deltas gives the keys back */
        uint64_t preKey = lo;
        for (uint64_t i = 0; i < count; ++i) {
            uint32_t flag = (uint32_t)get_bits(blob, flag_pos + (uint64_t)l * i, l);
            uint64_t delta = get_bits(blob, delta_pos, widths[flag]);
            delta_pos += widths[flag];
            if (i > 0 && delta == 0) return FSGO_DEC_BAD_KEY;
            uint64_t key = preKey + delta;
            if (key >= hi) return FSGO_DEC_BAD_KEY;
            preKey = key;
            int rc = sink(ctx, key, blob[i]);
            if (rc) return rc;
        }
        expect_off = next_off;
    }
    return FSGO_OK;
}

typedef struct { uint64_t *keys; int32_t *codes; uint64_t count; uint64_t limit; } parse_ctx;

static int parse_sink(void *vctx, uint64_t key, uint8_t code_byte)
{
    parse_ctx *c = (parse_ctx *)vctx;
    if (c->count >= c->limit) return FSGO_DEC_BAD_DIRECTORY;   /* more keys than the header's d */
    c->keys[c->count] = key;
    c->codes[c->count] = fsgo_code_from_byte(code_byte);
    c->count++;
    return 0;
}

int fsgo_parse(const uint8_t *stream, uint64_t bytes, uint64_t n, const fsgo_params *p,
               uint64_t *keys, int32_t *codes, uint64_t *d, double *sum)
{
    parse_ctx c; c.keys = keys; c.codes = codes; c.count = 0;
    c.limit = (bytes >= FSGO_HEADER) ? get_u64(stream + 24) : 0;
    int rc = walk_stream(stream, bytes, n, p, NULL, sum, parse_sink, &c);
    *d = c.count;
    return rc;
}

typedef struct { float *dense; float value[129]; uint32_t tau; } acc_ctx;

static int acc_sink(void *vctx, uint64_t key, uint8_t code_byte)
{
    acc_ctx *c = (acc_ctx *)vctx;
    uint32_t L = (uint32_t)(code_byte & 0x7Fu) + 1u;
    if (L > c->tau) return FSGO_DEC_BAD_CODE;
    /* phases 3-4: R^ = b^L, v^ = sum / R^ = B[L], sign from the code */
    float vhat = (code_byte & 0x80u) ? -c->value[L] : c->value[L];
    c->dense[key] = c->dense[key] + vhat;
    return 0;
}

int fsgo_decompress_accumulate(const uint8_t *stream, uint64_t bytes, uint64_t n,
                               const fsgo_params *p, float *dense)
{
    if (!params_ok(p) || n == 0) return FSGO_BAD_PARAM;
    acc_ctx c; c.dense = dense; c.tau = p->tau;
    if (bytes >= FSGO_HEADER) {
        double P[129], B[129];
        fsgo_tables(get_f64(stream + 40), p->base, p->tau, P, B);
        for (uint32_t k = 0; k <= p->tau; ++k) c.value[k] = (float)B[k];
    }
    return walk_stream(stream, bytes, n, p, NULL, NULL, acc_sink, &c);
}

/* ---------------------------------------------------------- model update */

int fsgo_sparse_adam_update(const uint8_t *const *streams, const uint64_t *bytes,
                            uint32_t num_streams, uint64_t n, const fsgo_params *p,
                            const fsgo_adam *h, float *theta, float *m, float *v)
{
    if (!params_ok(p) || n == 0) return FSGO_BAD_PARAM;
    float *g = (float *)calloc(n, sizeof(float));
    if (!g) return FSGO_BAD_PARAM;
    /* the aggregated gradient: the workers' decoded streams added up in order */
    for (uint32_t w = 0; w < num_streams; ++w) {
        int rc = fsgo_decompress_accumulate(streams[w], bytes[w], n, p, g);
        if (rc) { free(g); return rc; }
    }
    const float one_m_b1 = 1.0f - h->beta1, one_m_b2 = 1.0f - h->beta2;
    for (uint64_t k = 0; k < n; ++k) {
        const float gk = g[k];
        if (gk == 0.0f) continue;
        const float a1 = h->beta1 * m[k], a2 = one_m_b1 * gk;
        const float mk = a1 + a2;
        const float g2 = gk * gk;
        const float c1 = h->beta2 * v[k], c2 = one_m_b2 * g2;
        const float vk = c1 + c2;
        const float den = sqrtf(vk + h->eps);
        const float step = h->lr / den;
        const float upd = step * mk;
        m[k] = mk;
        v[k] = vk;
        theta[k] = theta[k] - upd;
    }
    free(g);
    return FSGO_OK;
}

/* ------------------------------------------------------- key-value input */

int fsgo_compress_kv(const uint64_t *keys, const float *values, uint64_t count,
                     uint64_t n, const fsgo_params *p, uint8_t *out, uint64_t cap,
                     uint64_t *total)
{
    if (n == 0) return FSGO_BAD_PARAM;
    for (uint64_t j = 0; j < count; ++j)
        if (keys[j] >= n || (j && keys[j] <= keys[j - 1])) return FSGO_BAD_PARAM;
    float *dense = (float *)calloc(n, sizeof(float));
    if (!dense) return FSGO_BAD_PARAM;
    for (uint64_t j = 0; j < count; ++j) dense[keys[j]] = values[j];
    int rc = fsgo_compress(dense, n, p, out, cap, total);
    free(dense);
    return rc;
}
