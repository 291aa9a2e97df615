// Decoder (decoder phases 1-4) and aggregation, for one stream or for several workers' streams
// of the same gradient in one launch.
//
// Phase 1: the length flags give every delta's width; an exclusive scan of the widths gives
// its bit offset.  Phase 2: an inclusive scan of the deltas, started at g*T, gives the keys
// back.  Phases 3-4: code L -> sum / b^L (the boundary B_L rounded to fp32), signed.  The
// aggregation adds the value into dense_out[key].  Keys are unique within a stream, and the
// streams of one launch are applied to a group in their given order by the same warp or block,
// so the read-modify-write needs no atomics and the result equals that of one call per stream.
//
// Work split: a group whose streams all hold few keys is decoded by one warp, any other by the
// whole block; either way a thread owns a run of consecutive keys, so that the scans are one
// shuffle scan (plus one shared-memory step for the block) per group, and a group is validated
// in full before any of it is applied.  The blobs of all streams of a group are first copied
// into shared memory with coalesced loads (one memory round trip for all of them), then parsed
// from there.
#pragma once

#include <cstddef>

#include "common.cuh"
#include "bits.cuh"
#include "compress.cuh"     // mbarrier / bulk-copy primitives

namespace fsg {

constexpr int      kDecThreads     = 256;
constexpr int      kDecWarps       = kDecThreads / 32;
constexpr int      kDecMaxStreams  = 8;       // streams per launch
constexpr uint32_t kDecWarpMax     = 256;     // groups with more keys (in any stream) go to the whole block (128 with more than two streams)
constexpr uint32_t kDecWarpSide    = 128;     // up to this many keys per stream a warp parses the streams side by side
constexpr int      kDecListMax     = 512;     // groups one block may own
constexpr uint32_t kWarpStageWords = 2048;    // >= kDecMaxStreams * ceil(kDecWarpMax * (8 + 5 + 14) / 32); 8 warps x 8 KiB = the tile's 64 KiB
constexpr uint32_t kBlockStageWords = 10240;  // blobs larger than this in total are parsed from global memory
constexpr uint32_t kDecSpinLimit   = 1u << 20;

struct DecArgs {
    const uint8_t*      stream[kDecMaxStreams];
    uint64_t            bytes[kDecMaxStreams];
    uint64_t            n;
    float*              dense;
    unsigned long long* status;     // sticky minimum of (group << 32 | key index << 8 | status)
    unsigned int*       q_ctl;      // {pushed, taken, done, exited, reserved}: queue of groups for whole blocks, shared by the grid
    unsigned int*       q_list;     // its G slots
    unsigned long long* trace;      // per-block stamps (only written by builds with -DFASTSGD_TRACE)
    double              base;
    uint32_t            W;          // streams in this launch
    uint32_t            G;
    uint32_t            tau;
    uint32_t            l;
    uint32_t            group_log2;
    uint32_t            spin_limit; // polls before a wait on the queue of large groups gives up (kDecSpinLimit unless a test shortens it)
    uint32_t            try_limit;  // tries before a wait on a bulk copy gives up
    // model update on the decoded coordinates (second pass; `dense` then holds the aggregated gradient)
    float*              theta;
    float*              m;
    float*              v;
    float               lr, beta1, beta2, eps;
};

// Modes of the decoder (template parameter MODE): 0 aggregation; 1 model update as a pass of its own; 2 both in one
// launch; 3 both in one launch on the packed state (theta, m, v, g per coordinate, g where dense_out[i] would be);
// 4 and 5: what 0 and 1 are to 2, for 3 (a group whose streams do not fit one decode_multi call).
__host__ __device__ constexpr bool mode_packed(int mode) { return mode >= 3; }
__host__ __device__ constexpr bool mode_fused(int mode) { return mode == 2 || mode == 3; }
__host__ __device__ constexpr int mode_apply(int mode) { return (mode == 1 || mode == 5) ? 1 : 0; }       // what apply_run does in the first sweep
// index of coordinate k's entry of dense_out (g) as a float
template <int MODE> __device__ __forceinline__ uint32_t dense_at(uint32_t k) { return mode_packed(MODE) ? 4u * k + 3u : k; }

// What a thread's run of K decoded (key, value) pairs does to the entries `cur` of dense_out at those keys
// (distinct; 0xFFFFFFFF: no key); the results are stored there by the caller.
// MODE 0: aggregation, cur + value.  MODE 1: model update: `cur` is the aggregated gradient g at that
// key, left there by an aggregation pass over the same streams; where it is non-zero the coordinate takes one
// Adam step (the experimental set-up's equations, no bias correction; one IEEE fp32 operation at a
// time) and g returns to zero, so that a key that several streams hold is updated once.  All loads of
// the moments and the parameters are issued before the first of them is needed.
// PACKED: the model's state is one array of (theta, m, v, g) per coordinate (dense_out points at it): one 16-byte
// load and one 16-byte store per updated coordinate instead of three sectors read and written.
template <int MODE, int K, bool PACKED = false>
__device__ __forceinline__ void apply_run(const DecArgs& a, const uint32_t (&kk)[K], const float (&cur)[K],
                                          const float (&value)[K], float (&res)[K]) {
    if (MODE == 0) {
#pragma unroll
        for (int k = 0; k < K; ++k) res[k] = __fadd_rn(cur[k], value[k]);
        return;
    }
    if constexpr (PACKED) {
        float4* state = reinterpret_cast<float4*>(a.dense);
        float4 st[K];
#pragma unroll
        for (int k = 0; k < K; ++k) {
            const bool on = kk[k] != 0xFFFFFFFFu && cur[k] != 0.0f;
            st[k] = on ? state[kk[k]] : make_float4(0.f, 0.f, 0.f, 0.f);
        }
#pragma unroll
        for (int k = 0; k < K; ++k) {
            if (kk[k] != 0xFFFFFFFFu && cur[k] != 0.0f) {
                const float mk = __fadd_rn(__fmul_rn(a.beta1, st[k].y), __fmul_rn(__fsub_rn(1.0f, a.beta1), cur[k]));
                const float vk = __fadd_rn(__fmul_rn(a.beta2, st[k].z), __fmul_rn(__fsub_rn(1.0f, a.beta2), __fmul_rn(cur[k], cur[k])));
                const float step = __fdiv_rn(a.lr, __fsqrt_rn(__fadd_rn(vk, a.eps)));
                state[kk[k]] = make_float4(__fsub_rn(st[k].x, __fmul_rn(step, mk)), mk, vk, 0.0f);
            }
            res[k] = 0.0f;
        }
        return;
    }
    float pm[K], pv[K], pt[K];
#pragma unroll
    for (int k = 0; k < K; ++k) {
        const bool on = kk[k] != 0xFFFFFFFFu && cur[k] != 0.0f;
        pm[k] = on ? a.m[kk[k]] : 0.0f;
        pv[k] = on ? a.v[kk[k]] : 0.0f;
        pt[k] = on ? a.theta[kk[k]] : 0.0f;
    }
#pragma unroll
    for (int k = 0; k < K; ++k) {
        if (kk[k] != 0xFFFFFFFFu && cur[k] != 0.0f) {
            const float mk = __fadd_rn(__fmul_rn(a.beta1, pm[k]), __fmul_rn(__fsub_rn(1.0f, a.beta1), cur[k]));
            const float vk = __fadd_rn(__fmul_rn(a.beta2, pv[k]), __fmul_rn(__fsub_rn(1.0f, a.beta2), __fmul_rn(cur[k], cur[k])));
            const float step = __fdiv_rn(a.lr, __fsqrt_rn(__fadd_rn(vk, a.eps)));
            a.m[kk[k]] = mk;
            a.v[kk[k]] = vk;
            a.theta[kk[k]] = __fsub_rn(pt[k], __fmul_rn(step, mk));
        }
        res[k] = 0.0f;
    }
}

#ifdef FASTSGD_TRACE
__device__ __forceinline__ unsigned long long read_globaltimer_dec() {
    unsigned long long t;
    asm volatile("mov.u64 %0, %%globaltimer;" : "=l"(t));
    return t;
}
#define FSG_DEC_STAMP(var) do { if (tid == 0) var = read_globaltimer_dec(); } while (0)
#else
#define FSG_DEC_STAMP(var) do { } while (0)
#endif

__device__ __forceinline__ void dec_fail(const DecArgs& a, uint32_t g, uint32_t j, int st) {
    atomicMin(a.status, ((unsigned long long)g << 32) | ((unsigned long long)(j & 0xFFFFFFu) << 8) | (unsigned)st);
}

__device__ __forceinline__ int check_header(const DecArgs& a, uint64_t bytes, const uint32_t* w, uint64_t* total_out, double* sum_out) {
    if (w[0] != kMagic) return kStBadMagic;
    if (w[1] != kVersion) return kStBadVersion;
    if (w[2] != (uint32_t)kStOk) return kStBadStatus;
    const uint64_t n = (uint64_t)w[4] | ((uint64_t)w[5] << 32);
    if (n != a.n) return kStNMismatch;
    const unsigned long long bb = (unsigned long long)w[12] | ((unsigned long long)w[13] << 32);
    if (bb != (unsigned long long)__double_as_longlong(a.base) || w[3] != a.tau ||
        (w[14] & 0xFFu) != a.l || ((w[14] >> 8) & 0xFFu) != a.group_log2 || w[15] != a.G)
        return kStParamMismatch;
    const uint64_t total = (uint64_t)w[8] | ((uint64_t)w[9] << 32);
    const uint64_t fixed = (uint64_t)kHeaderBytes + 8ull * a.G;
    if (total > bytes || total < fixed || (total & 3ull)) return kStTruncated;
    *total_out = total;
    *sum_out = __longlong_as_double((long long)((unsigned long long)w[10] | ((unsigned long long)w[11] << 32)));
    return kStOk;
}

struct DecShared {
    float              val[kDecMaxStreams][132];
    double             sum[kDecMaxStreams];
    uint32_t           total_words[kDecMaxStreams];
    uint32_t           ok[kDecMaxStreams];
    uint32_t           scan[2][kDecWarps];
    uint32_t           scanm[2][4][kDecWarps];   // the same for up to four streams scanned together
    unsigned long long first_bad_m[4];
    uint32_t           big[kDecListMax];
    unsigned long long first_bad;     // min over threads of (key index << 8 | status), block path
    uint32_t           big_count;     // large groups this block has found among its own
    uint32_t           local_g;       // the first of them: decoded by this block itself, the others go to the queue
    unsigned long long tile_bar;      // mbarrier of the bulk copy that loads the tile
    // per stream, for the group the block works on
    uint32_t           g_count[kDecMaxStreams], g_M[kDecMaxStreams], g_off[kDecMaxStreams], g_nwords[kDecMaxStreams],
                       g_base[kDecMaxStreams], g_valid[kDecMaxStreams];
    uint32_t           bstage[kBlockStageWords];
    union alignas(128) {               // (bulk copies need 16-byte aligned shared addresses)
        uint32_t       wstage[kDecWarps][kWarpStageWords];   // warp path: the streams' blobs of a small group
        float          tile[1u << 14];                       // block path: the group's slice of dense_out
    } u;
};
static_assert(sizeof(DecShared) <= 113 * 1024, "two blocks per SM");
static_assert(offsetof(DecShared, u) % 128 == 0, "tile alignment");

// bits [pos, pos+nb) of a most-significant-bit-first sequence held as little-endian 32-bit words
// (shared or global memory); nb <= 32
__device__ __forceinline__ uint32_t get_bits(const uint32_t* words, uint32_t nwords, uint32_t pos, uint32_t nb) {
    const uint32_t wi = pos >> 5, sh = pos & 31u;
    const uint32_t w0 = wi < nwords ? bswap32(words[wi]) : 0u;
    const uint32_t w1 = (wi + 1u) < nwords ? bswap32(words[wi + 1u]) : 0u;
    const unsigned long long both = ((unsigned long long)w0 << 32) | w1;
    if (nb == 0) return 0u;
    return (uint32_t)((both >> (64u - sh - nb)) & ((nb >= 32u) ? 0xFFFFFFFFull : ((1ull << nb) - 1ull)));
}

// exclusive scan of one value per thread over the warp (BLOCK = false) or the block; also returns the
// total.  `which` alternates between the two shared arrays so that one barrier per scan is enough.
template <bool BLOCK>
__device__ __forceinline__ uint32_t excl_scan(uint32_t v, uint32_t* total, DecShared& s, int lane, int warp, int which) {
    const uint32_t incl = warp_incl_scan(v, lane);
    if (!BLOCK) {
        *total = __shfl_sync(kFullMask, incl, 31);
        return incl - v;
    }
    if (lane == 31) s.scan[which][warp] = incl;
    __syncthreads();
    uint32_t before = 0, all = 0;
#pragma unroll
    for (int w = 0; w < kDecWarps; ++w) {
        const uint32_t t = s.scan[which][w];
        if (w < warp) before += t;
        all += t;
    }
    *total = all;
    return before + incl - v;
}

// Directory entry of group g in one stream, checked.  Returns false (and records the status) if
// it is inconsistent.  count = 0 for an empty group.
__device__ __forceinline__ bool read_dir(const DecArgs& a, const uint32_t* sw, uint32_t g, uint32_t total_words,
                                         uint32_t* count, uint32_t* M, uint32_t* off, uint32_t* nwords) {
    const uint32_t fixed_words = (kHeaderBytes + 8u * a.G) >> 2;
    const uint32_t* dir = sw + (kHeaderBytes >> 2);
    const uint32_t e0 = __ldg(dir + 2 * g), o = __ldg(dir + 2 * g + 1);
    const uint32_t next_off = (g + 1 < a.G) ? __ldg(dir + 2 * g + 3) : total_words;
    const uint32_t c = e0 & 0xFFFFFFu, m = e0 >> 24;
    *count = 0; *M = m; *off = o; *nwords = 0;
    if ((g == 0 && o != fixed_words) || next_off < o || next_off > total_words || o < fixed_words) {
        dec_fail(a, g, 0u, kStBadDirectory);
        return false;
    }
    if (c == 0) {
        if (e0 != 0u || next_off != o) { dec_fail(a, g, 0u, kStBadDirectory); return false; }
        return true;
    }
    const uint64_t lo64 = (uint64_t)g << a.group_log2;
    const uint64_t hi64 = lo64 + (1ull << a.group_log2);
    const uint32_t span = (uint32_t)((hi64 < a.n ? hi64 : a.n) - lo64);
    const uint32_t nw = next_off - o;
    // (a blob is never longer than count * (8 + l + M) bits rounded up to words: also bounds the staging copy)
    if (c > span || m < 1u || m > a.group_log2 || (uint64_t)(8u + a.l) * c > 32ull * nw ||
        (uint64_t)nw > ((uint64_t)c * (8u + a.l + m) + 31ull) / 32ull) {
        dec_fail(a, g, 0u, kStBadDirectory);
        return false;
    }
    *count = c; *nwords = nw;
    return true;
}

// Sequential reader of a most-significant-bit-first sequence held as little-endian 32-bit words: fields of up to 32
// bits, one after the other, from a 64-bit window that is topped up a word at a time (beyond nwords: zeros).
struct BitReader {
    const uint32_t*    w;
    uint32_t           nwords, next;
    unsigned long long buf;          // the next `avail` bits of the sequence, left-aligned; avail > 32 between calls
    int                avail;
    __device__ __forceinline__ void init(const uint32_t* words, uint32_t nw, uint32_t pos) {
        w = words; nwords = nw;
        const uint32_t wi = pos >> 5, sh = pos & 31u;
        const uint32_t w0 = wi < nw ? bswap32(words[wi]) : 0u, w1 = (wi + 1u) < nw ? bswap32(words[wi + 1u]) : 0u;
        buf = ((((unsigned long long)w0) << 32) | w1) << sh;
        avail = 64 - (int)sh;
        next = wi + 2u;
    }
    __device__ __forceinline__ uint32_t take(uint32_t nb) {
        const uint32_t v = nb ? (uint32_t)(buf >> (64u - nb)) : 0u;
        buf <<= nb;
        avail -= (int)nb;
        if (avail <= 32) {
            const uint32_t x = next < nwords ? bswap32(w[next]) : 0u;
            buf |= (unsigned long long)x << (32 - avail);
            avail += 32;
            ++next;
        }
        return v;
    }
};

// The four code bytes j, j+1, j+2, j+3 of a blob (byte i in bits 8i.. of the result); two word loads.
__device__ __forceinline__ uint32_t codes4(const uint32_t* blob, uint32_t nwords, uint32_t j) {
    const uint32_t wi = j >> 2;
    const uint32_t w0 = wi < nwords ? blob[wi] : 0u, w1 = (wi + 1u) < nwords ? blob[wi + 1u] : 0u;
    return __funnelshift_r(w0, w1, 8u * (j & 3u));
}

// One group of one stream with any number of keys, decoded by the whole block in rounds of 8 keys per thread: a
// round's flags, widths, deltas and keys stay in registers (one block scan of the widths and one of the deltas per
// round); the bit position of the next delta and the last key carry over.  A round is validated in full before it is
// applied; the blob's length, which the flags of ALL rounds imply, is checked when the last round is done.  With
// `tile` the values go into the group's slice of dense_out held in shared memory, else straight into dense_out.
template <int MODE>
__device__ __forceinline__ void decode_long(const DecArgs& a, DecShared& s, const uint32_t* blob, uint32_t nwords,
                                            uint32_t g, uint32_t count, uint32_t M, const float* val, float* tile,
                                            int t, int nthreads, int lane, int warp) {
    constexpr int KMAX = 8;
    const uint64_t lo64 = (uint64_t)g << a.group_log2;
    const uint64_t hi64 = lo64 + (1ull << a.group_log2);
    const uint32_t lo = (uint32_t)lo64;
    const uint32_t hi = (uint32_t)(hi64 < a.n ? hi64 : a.n);
    const uint32_t levels_m1 = (1u << a.l) - 1u;
    const uint32_t flag_pos0 = 8u * count;
    const uint32_t delta_pos0 = flag_pos0 + a.l * count;
    const uint32_t per_round = (uint32_t)KMAX * (uint32_t)nthreads;
    uint32_t bitpos = delta_pos0, keybase = lo;
    bool failed = false;                                  // uniform over the block
    for (uint32_t r0 = 0; r0 < count; r0 += per_round) {
        const uint32_t rc = min(per_round, count - r0);
        const uint32_t K = (rc + nthreads - 1) / nthreads;
        const uint32_t jb = r0 + min(rc, (uint32_t)t * K), je = r0 + min(rc, (uint32_t)t * K + K);
        uint32_t wv[KMAX], dv[KMAX], codes[2], wsum = 0u;
#pragma unroll
        for (int k0 = 0; k0 < KMAX; k0 += 4) {
            const uint32_t fb = (jb + k0 < je) ? get_bits(blob, nwords, flag_pos0 + a.l * (jb + k0), a.l * 4u) : 0u;
#pragma unroll
            for (int k = k0; k < k0 + 4; ++k) {
                const uint32_t f = (fb >> (a.l * (uint32_t)(k0 + 3 - k))) & levels_m1;
                wv[k] = (jb + k < je) ? ((f + 1u) * M + levels_m1) >> a.l : 0u;
                wsum += wv[k];
            }
        }
        codes[0] = codes4(blob, nwords, jb);
        codes[1] = codes4(blob, nwords, jb + 4u);
        uint32_t wtotal, dtotal;
        const uint32_t pos0 = bitpos + excl_scan<true>(wsum, &wtotal, s, lane, warp, 0);
        if (failed) {                                     // only the blob's length is still of interest
            bitpos = min(bitpos + wtotal, 0xFFF00000u);
            __syncthreads();                              // (the scan's scratch is rewritten next round)
            continue;
        }
        BitReader rd;
        rd.init(blob, nwords, pos0);
        uint32_t dsum = 0u;
#pragma unroll
        for (int k = 0; k < KMAX; ++k) {
            dv[k] = rd.take(wv[k]);
            dsum = min(dsum + dv[k], 1u << 21);
        }
        const uint32_t key0 = keybase + excl_scan<true>(dsum, &dtotal, s, lane, warp, 1);
        unsigned long long bad = ~0ull;
        {
            uint32_t key = key0;
#pragma unroll
            for (int k = 0; k < KMAX; ++k) {
                const uint32_t j = jb + k;
                if (j < je && bad == ~0ull) {
                    key += dv[k];
                    const uint32_t code = (codes[k >> 2] >> (8u * (uint32_t)(k & 3))) & 0xFFu;
                    if ((j > 0 && dv[k] == 0u) || key >= hi || key < lo) bad = ((unsigned long long)j << 8) | (unsigned)kStBadKey;
                    else if ((code & 0x7Fu) + 1u > a.tau) bad = ((unsigned long long)j << 8) | (unsigned)kStBadCode;
                }
            }
        }
        if (__syncthreads_or(bad != ~0ull)) {             // one barrier when the round is sound
            if (t == 0) s.first_bad = ~0ull;
            __syncthreads();
            if (bad != ~0ull) atomicMin(&s.first_bad, bad);
            __syncthreads();
            bad = s.first_bad;
            __syncthreads();
            if (t == 0) dec_fail(a, g, (uint32_t)(bad >> 8), (int)(bad & 0xFFull));
            // nothing more is applied; the remaining rounds only add up the widths, since a blob whose length disagrees
            // with its flags is reported as that (key index 0: it takes precedence in the status word)
            failed = true;
            bitpos = min(bitpos + wtotal, 0xFFF00000u);
            continue;
        }
        {
            uint32_t key = key0;
            uint32_t kk[KMAX]; float vv[KMAX], dd[KMAX], res[KMAX];
#pragma unroll
            for (int k = 0; k < KMAX; ++k) {
                kk[k] = 0xFFFFFFFFu; vv[k] = 0.f;
                if (jb + k < je) {
                    key += dv[k];
                    const uint32_t code = (codes[k >> 2] >> (8u * (uint32_t)(k & 3))) & 0xFFu;
                    const float mag = val[(code & 0x7Fu) + 1u];
                    kk[k] = key; vv[k] = (code & 0x80u) ? -mag : mag;
                }
            }
            if (tile != nullptr) {
#pragma unroll
                for (int k = 0; k < KMAX; ++k) dd[k] = kk[k] != 0xFFFFFFFFu ? tile[kk[k] - lo] : 0.f;
                apply_run<MODE, KMAX>(a, kk, dd, vv, res);
#pragma unroll
                for (int k = 0; k < KMAX; ++k) if (kk[k] != 0xFFFFFFFFu) tile[kk[k] - lo] = res[k];
            } else {
#pragma unroll
                for (int k = 0; k < KMAX; ++k) dd[k] = kk[k] != 0xFFFFFFFFu ? a.dense[kk[k]] : 0.f;
                apply_run<MODE, KMAX>(a, kk, dd, vv, res);
#pragma unroll
                for (int k = 0; k < KMAX; ++k) if (kk[k] != 0xFFFFFFFFu) a.dense[kk[k]] = res[k];
            }
        }
        bitpos = min(bitpos + wtotal, 0xFFF00000u);
        keybase = min(keybase + dtotal, 0xFFF00000u);     // (saturate only when already invalid)
    }
    if ((((uint64_t)bitpos + 31ull) >> 5) != nwords && t == 0) dec_fail(a, g, 0u, kStBadDirectory);
}

// Exclusive scans of NS values per thread at once (one barrier for all of them in a block).
template <bool BLOCK, int NS>
__device__ __forceinline__ void excl_scan_multi(const uint32_t (&v)[NS], uint32_t (&excl)[NS], uint32_t (&total)[NS],
                                                DecShared& s, int lane, int warp, int which) {
    uint32_t incl[NS];
#pragma unroll
    for (int w = 0; w < NS; ++w) incl[w] = warp_incl_scan(v[w], lane);
    if (!BLOCK) {
#pragma unroll
        for (int w = 0; w < NS; ++w) { total[w] = __shfl_sync(kFullMask, incl[w], 31); excl[w] = incl[w] - v[w]; }
        return;
    }
    if (lane == 31) {
#pragma unroll
        for (int w = 0; w < NS; ++w) s.scanm[which][w][warp] = incl[w];
    }
    __syncthreads();
#pragma unroll
    for (int w = 0; w < NS; ++w) {
        uint32_t before = 0, all = 0;
#pragma unroll
        for (int k = 0; k < kDecWarps; ++k) {
            const uint32_t t = s.scanm[which][w][k];
            if (k < warp) before += t;
            all += t;
        }
        total[w] = all;
        excl[w] = before + incl[w] - v[w];
    }
}

// One group of NS streams, decoded together by a warp (BLOCK = false) or by the block: the streams
// are parsed side by side (independent dependency chains, one scan barrier for all of them), each
// is validated completely, and the sound ones are applied in stream order.  Every stream holds at
// most KMAX * nthreads keys, so a thread's run of consecutive keys stays in registers.
template <int MODE, bool BLOCK, int NS, int KMAX, bool TWO_GROUPS = false>
__device__ __forceinline__ void decode_multi(const DecArgs& a, DecShared& s, const uint32_t* const (&blob)[NS],
                                             const uint32_t (&nwords)[NS], const uint32_t (&count)[NS], const uint32_t (&M)[NS],
                                             const float* const (&val)[NS], uint32_t g, float* tile,
                                             int t, int nthreads, int lane, int warp, uint32_t g_other = 0xFFFFFFFFu) {
    // (g_other: slots 1.. hold another group of the same stream instead of other streams of group g)
    uint32_t gs[NS], lo[NS], hi[NS];
#pragma unroll
    for (int w = 0; w < NS; ++w) {
        gs[w] = (w == 0 || !TWO_GROUPS) ? g : g_other;
        const uint64_t lo64 = (uint64_t)gs[w] << a.group_log2;
        const uint64_t hi64 = lo64 + (1ull << a.group_log2);
        lo[w] = (uint32_t)lo64;
        hi[w] = (uint32_t)(hi64 < a.n ? hi64 : a.n);
    }
    const bool lead = (t == 0);
    const uint32_t levels_m1 = (1u << a.l) - 1u;
    uint32_t jb[NS], je[NS], wv[NS][KMAX], dv[NS][KMAX];
    bool live[NS];                                    // uniform: the stream has keys here and has not failed a check

    // phase 1: widths from the flags; their sum fixes the blob's length, which must be the directory's
    uint32_t wsum[NS], pos0[NS], wtotal[NS];
#pragma unroll
    for (int w = 0; w < NS; ++w) {
        live[w] = count[w] != 0u;
        const uint32_t K = (count[w] + nthreads - 1) / nthreads;
        jb[w] = min(count[w], (uint32_t)t * K); je[w] = min(count[w], jb[w] + K);
        const uint32_t flag_pos0 = 8u * count[w];
        wsum[w] = 0u;
#pragma unroll
        for (int k = 0; k < KMAX; ++k) {
            wv[w][k] = 0u;
            if (jb[w] + k < je[w]) {
                const uint32_t f = get_bits(blob[w], nwords[w], flag_pos0 + a.l * (jb[w] + k), a.l);
                wv[w][k] = ((f + 1u) * M[w] + levels_m1) >> a.l;
            }
            wsum[w] += wv[w][k];
        }
    }
    excl_scan_multi<BLOCK, NS>(wsum, pos0, wtotal, s, lane, warp, 0);
#pragma unroll
    for (int w = 0; w < NS; ++w) {
        const uint32_t delta_pos0 = (8u + a.l) * count[w];
        pos0[w] += delta_pos0;
        if (live[w] && (((uint64_t)delta_pos0 + wtotal[w] + 31ull) >> 5) != nwords[w]) {
            if (lead) dec_fail(a, gs[w], 0u, kStBadDirectory);
            live[w] = false;
        }
    }

    // phase 2: this thread's deltas and their sum, then the key before its first one
    uint32_t dsum[NS], key0[NS], dtotal[NS];
#pragma unroll
    for (int w = 0; w < NS; ++w) {
        uint32_t pos = pos0[w];
        dsum[w] = 0u;
#pragma unroll
        for (int k = 0; k < KMAX; ++k) {
            dv[w][k] = live[w] ? get_bits(blob[w], nwords[w], pos, wv[w][k]) : 0u;     // width 0 beyond the run: reads as 0
            pos += wv[w][k];
            dsum[w] = min(dsum[w] + dv[w][k], 1u << 21);                               // saturates only when already invalid
        }
    }
    excl_scan_multi<BLOCK, NS>(dsum, key0, dtotal, s, lane, warp, 1);

    // validation of each stream's whole group before anything of it is applied: first key index that
    // repeats, leaves the group, or carries a code beyond tau
    unsigned long long bad[NS];
    bool any_bad = false;
#pragma unroll
    for (int w = 0; w < NS; ++w) {
        key0[w] += lo[w];
        bad[w] = ~0ull;
        uint32_t key = key0[w];
#pragma unroll
        for (int k = 0; k < KMAX; ++k) {
            const uint32_t j = jb[w] + k;
            if (live[w] && j < je[w] && bad[w] == ~0ull) {
                key += dv[w][k];
                const uint32_t code = (blob[w][j >> 2] >> (8u * (j & 3u))) & 0xFFu;
                if ((j > 0 && dv[w][k] == 0u) || key >= hi[w]) bad[w] = ((unsigned long long)j << 8) | (unsigned)kStBadKey;
                else if ((code & 0x7Fu) + 1u > a.tau) bad[w] = ((unsigned long long)j << 8) | (unsigned)kStBadCode;
            }
        }
        any_bad = any_bad || bad[w] != ~0ull;
    }
    if (BLOCK) {
        if (__syncthreads_or(any_bad ? 1 : 0)) {          // one barrier when every stream is sound
            if (t < NS) s.first_bad_m[t] = ~0ull;
            __syncthreads();
#pragma unroll
            for (int w = 0; w < NS; ++w) if (bad[w] != ~0ull) atomicMin(&s.first_bad_m[w], bad[w]);
            __syncthreads();
#pragma unroll
            for (int w = 0; w < NS; ++w) bad[w] = s.first_bad_m[w];
            __syncthreads();
        }
    } else if (__any_sync(kFullMask, any_bad)) {
#pragma unroll
        for (int w = 0; w < NS; ++w) {
            const uint32_t blo = __reduce_min_sync(kFullMask, (uint32_t)(bad[w] < 0xFFFFFFFFull ? bad[w] : 0xFFFFFFFFull));
            bad[w] = blo == 0xFFFFFFFFu ? ~0ull : (unsigned long long)blo;
        }
    }
#pragma unroll
    for (int w = 0; w < NS; ++w)
        if (live[w] && bad[w] != ~0ull) {
            if (lead) dec_fail(a, gs[w], (uint32_t)(bad[w] >> 8), (int)(bad[w] & 0xFFull));
            live[w] = false;
        }

    // phases 3-4 and the aggregation, stream by stream
    bool first = true;
#pragma unroll
    for (int w = 0; w < NS; ++w) {
        if (!live[w]) continue;
        if (!first) { if (BLOCK) __syncthreads(); else __syncwarp(); }    // the stream before may hold the same keys
        first = false;
        uint32_t key = key0[w];
        uint32_t kk[KMAX]; float vv[KMAX];
#pragma unroll
        for (int k = 0; k < KMAX; ++k) {
            const uint32_t j = jb[w] + k;
            kk[k] = 0xFFFFFFFFu; vv[k] = 0.f;
            if (j < je[w]) {
                key += dv[w][k];
                const uint32_t code = (blob[w][j >> 2] >> (8u * (j & 3u))) & 0xFFu;
                const float mag = val[w][(code & 0x7Fu) + 1u];
                kk[k] = key; vv[k] = (code & 0x80u) ? -mag : mag;
            }
        }
        float dd[KMAX], res[KMAX];                             // distinct keys: all loads, then all stores
        if (BLOCK && tile != nullptr) {
#pragma unroll
            for (int k = 0; k < KMAX; ++k) dd[k] = kk[k] != 0xFFFFFFFFu ? tile[kk[k] - lo[w]] : 0.f;
            apply_run<mode_apply(MODE), KMAX, mode_packed(MODE)>(a, kk, dd, vv, res);
#pragma unroll
            for (int k = 0; k < KMAX; ++k) if (kk[k] != 0xFFFFFFFFu) tile[kk[k] - lo[w]] = res[k];
        } else {
#pragma unroll
            for (int k = 0; k < KMAX; ++k) dd[k] = kk[k] != 0xFFFFFFFFu ? a.dense[dense_at<MODE>(kk[k])] : 0.f;
            apply_run<mode_apply(MODE), KMAX, mode_packed(MODE)>(a, kk, dd, vv, res);
#pragma unroll
            for (int k = 0; k < KMAX; ++k) if (kk[k] != 0xFFFFFFFFu) a.dense[dense_at<MODE>(kk[k])] = res[k];
        }
    }

    // MODE 2 (the caller has given every stream of the group in this one call; dense_out in global memory):
    // the model update from the same keys, still in registers.  Every key's aggregated g is taken out of
    // dense_out by an atomic exchange with 0: of the streams that hold a key the one that gets there first
    // receives g and updates the coordinate, the others receive 0 (whichever it is, the result is the same);
    // no stream waits for another, and all the exchanges are in flight together.
    if constexpr (mode_fused(MODE)) {
        static_assert(!BLOCK, "the block path updates from its slice in shared memory");
        if (first) return;                                     // (uniform) nothing was applied
        __syncwarp();
        constexpr int KA = NS * KMAX;
        uint32_t ka[KA]; float ga[KA];
#pragma unroll
        for (int w = 0; w < NS; ++w) {
            uint32_t key = key0[w];
#pragma unroll
            for (int k = 0; k < KMAX; ++k) {
                const bool on = live[w] && jb[w] + k < je[w];
                key += dv[w][k];
                ka[w * KMAX + k] = on ? key : 0xFFFFFFFFu;
            }
        }
#pragma unroll
        for (int i = 0; i < KA; ++i) ga[i] = ka[i] != 0xFFFFFFFFu ? atomicExch(a.dense + dense_at<MODE>(ka[i]), 0.0f) : 0.0f;
        constexpr int KB = KA < 8 ? KA : 8;                    // moments and parameters of eight keys loaded at a time
#pragma unroll
        for (int i0 = 0; i0 < KA; i0 += KB) {
            uint32_t kb[KB]; float gb[KB], vb[KB], rb[KB];
#pragma unroll
            for (int i = 0; i < KB; ++i) { kb[i] = ka[i0 + i]; gb[i] = ga[i0 + i]; vb[i] = 0.0f; }
            apply_run<1, KB, mode_packed(MODE)>(a, kb, gb, vb, rb);
        }
    }
}

// Copies a blob of nw words into shared memory: all of a lane's loads (up to four) in flight before its stores.
__device__ __forceinline__ void stage_blob(uint32_t* dst, const uint32_t* src, uint32_t nw, int lane) {
    for (uint32_t i0 = 0; i0 < nw; i0 += 128u) {
        uint32_t r[4];
#pragma unroll
        for (int u = 0; u < 4; ++u) {
            const uint32_t i = i0 + (uint32_t)u * 32u + (uint32_t)lane;
            r[u] = i < nw ? __ldg(src + i) : 0u;
        }
#pragma unroll
        for (int u = 0; u < 4; ++u) {
            const uint32_t i = i0 + (uint32_t)u * 32u + (uint32_t)lane;
            if (i < nw) dst[i] = r[u];
        }
    }
}

// The warp path's decode of one small group whose blobs are staged (lane w holds stream w's directory
// fields): up to four streams at a time, parsed side by side and applied in stream order.  DM: what
// decode_multi does with the values (0, 1, or 2 = both when W <= 4 puts every stream in the one call).
// Used by the kernel's mode 2 only: modes 0 and 1 keep the same loop in the kernel's body, where the
// compiler's code for it measured 15 % faster on four sparse streams than through this function.
template <int DM>
__device__ __forceinline__ void warp_fours(const DecArgs& a, DecShared& s, const uint32_t* stage, uint32_t count, uint32_t M,
                                           uint32_t base, uint32_t nwords, uint32_t W, uint32_t g, int lane, int warp) {
    for (uint32_t w0 = 0; w0 < W; w0 += 4u) {
        const uint32_t ns = W - w0 < 4u ? W - w0 : 4u;
        const uint32_t* bl[4]; uint32_t nwv[4], cv[4], mv[4]; const float* vl[4];
#pragma unroll
        for (int i = 0; i < 4; ++i) {
            const uint32_t src = (uint32_t)i < ns ? w0 + i : w0;
            const uint32_t c = __shfl_sync(kFullMask, count, src), b = __shfl_sync(kFullMask, base, src);
            nwv[i] = __shfl_sync(kFullMask, nwords, src); mv[i] = __shfl_sync(kFullMask, M, src);
            cv[i] = (uint32_t)i < ns ? c : 0u;
            bl[i] = stage + b; vl[i] = s.val[src];
        }
        if (ns == 1u) {
            const uint32_t* b1[1] = {bl[0]}; const uint32_t n1[1] = {nwv[0]}, c1[1] = {cv[0]}, m1[1] = {mv[0]}; const float* v1[1] = {vl[0]};
            decode_multi<DM, false, 1, 4>(a, s, b1, n1, c1, m1, v1, g, nullptr, lane, 32, lane, warp);
        } else if (ns == 2u) {
            const uint32_t* b2[2] = {bl[0], bl[1]}; const uint32_t n2[2] = {nwv[0], nwv[1]}, c2[2] = {cv[0], cv[1]}, m2[2] = {mv[0], mv[1]};
            const float* v2[2] = {vl[0], vl[1]};
            decode_multi<DM, false, 2, 4>(a, s, b2, n2, c2, m2, v2, g, nullptr, lane, 32, lane, warp);
        } else {
            decode_multi<DM, false, 4, 4>(a, s, bl, nwv, cv, mv, vl, g, nullptr, lane, 32, lane, warp);
        }
        __syncwarp();          // these streams' stores before the next streams' loads of the same keys
    }
}

// A decode_multi call of the kernel below.  MODE 2 (aggregation and model update in one launch): `fused`
// when this call holds every stream of the group (both sweeps inside the call), else the caller's pass
// (0: aggregation over all the group's calls, then 1: the update over all of them again).
#define FSG_DECODE_MULTI(fused, B_, NS_, K_, TG_, ...)                                        \
    do {                                                                                      \
        if constexpr (mode_fused(MODE)) {                                                     \
            if (fused) decode_multi<MODE, B_, NS_, K_, TG_>(__VA_ARGS__);                     \
            else if (pass == 0) decode_multi<(MODE == 3 ? 4 : 0), B_, NS_, K_, TG_>(__VA_ARGS__);  \
            else decode_multi<(MODE == 3 ? 5 : 1), B_, NS_, K_, TG_>(__VA_ARGS__);            \
        } else {                                                                              \
            decode_multi<MODE, B_, NS_, K_, TG_>(__VA_ARGS__);                                \
        }                                                                                     \
    } while (0)

// (the same without the fused form: the block path, whose mode 2 keeps the slice of g in shared memory)
#define FSG_DECODE_MULTI_PASS(B_, NS_, K_, TG_, ...)                                          \
    do {                                                                                      \
        if constexpr (mode_fused(MODE)) {                                                     \
            if (pass == 0) decode_multi<(MODE == 3 ? 4 : 0), B_, NS_, K_, TG_>(__VA_ARGS__);  \
            else decode_multi<(MODE == 3 ? 5 : 1), B_, NS_, K_, TG_>(__VA_ARGS__);            \
        } else {                                                                              \
            decode_multi<MODE, B_, NS_, K_, TG_>(__VA_ARGS__);                                \
        }                                                                                     \
    } while (0)

// ONE_STREAM: the launch holds a single stream (its own instantiation, so that the code of the
// many-stream paths and of the two-groups-per-warp path do not weigh on each other)
// MODE: what a decoded value does to dense_out: 0 aggregation, 1 model update, 2 both, 3 both on the packed state (see mode_packed).
template <bool ONE_STREAM, int MODE = 0>
__global__ void __launch_bounds__(kDecThreads, 2)
k_decode_accumulate(const DecArgs a, const __grid_constant__ PowTable pw) {
    extern __shared__ __align__(128) unsigned char dec_smem_raw[];
    DecShared& s = *reinterpret_cast<DecShared*>(dec_smem_raw);
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const uint32_t W = ONE_STREAM ? 1u : a.W;         // (one stream: a constant, so that none of the many-stream code is compiled in)
#ifdef FASTSGD_TRACE
    // per-block %globaltimer stamps: start, tables ready, own groups done, end; groups taken from the queue
    unsigned long long T0 = 0, T1 = 0, T2 = 0; unsigned int taken = 0;
#endif
    FSG_DEC_STAMP(T0);

    if (tid == 0) {
        mbar_init(&s.tile_bar, 1u);
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
        s.big_count = 0u;
    }
    uint32_t tile_parity = 0;
    // ---- headers: thread w checks stream w
    if (tid < (int)W) {
        const uint32_t* sw = reinterpret_cast<const uint32_t*>(a.stream[tid]);
        uint32_t h[16];
#pragma unroll
        for (int i = 0; i < 16; ++i) h[i] = __ldg(sw + i);
        uint64_t total = 0; double S = 0.0;
        const int st = check_header(a, a.bytes[tid], h, &total, &S);
        s.ok[tid] = st == kStOk ? 1u : 0u;
        s.total_words[tid] = (uint32_t)(total >> 2);
        s.sum[tid] = S;
        if (st != kStOk && blockIdx.x == 0) dec_fail(a, 0u, 0u, st);
    }
    __syncthreads();
    // phases 3-4 as a table per stream: value[L] = (float)(sum / b^L)
    for (uint32_t idx = tid; idx < W * 132u; idx += kDecThreads) {
        const uint32_t w = idx / 132u, k = idx % 132u;
        if (k <= a.tau && s.ok[w]) s.val[w][k] = __double2float_rn(__ddiv_rn(s.sum[w], pw.P[k]));
    }
    __syncthreads();

    FSG_DEC_STAMP(T1);
    // ---- this block owns groups blockIdx.x, blockIdx.x + gridDim.x, ...; warp w takes every 8th of them
    // (a warp applies the streams of a group one after the other: with many streams the whole block is the better choice sooner)
    const uint32_t warp_max = W <= 2u ? kDecWarpMax : kDecWarpSide;
    if (ONE_STREAM) {
        // One stream: a warp takes its groups two at a time (lane 0: group g, lane 1: the warp's next
        // group), so that their directory reads, blob copies, parses and updates overlap.
        const uint32_t stride = kDecWarps * gridDim.x;
        const uint32_t* sw0 = reinterpret_cast<const uint32_t*>(a.stream[0]);
        for (uint32_t g = blockIdx.x + warp * gridDim.x; g < a.G; g += 2u * stride) {
            const uint32_t gl = g + (uint32_t)lane * stride;
            uint32_t count = 0, M = 0, off = 0, nwords = 0;
            if (lane < 2 && gl < a.G && s.ok[0]) read_dir(a, sw0, gl, s.total_words[0], &count, &M, &off, &nwords);
#pragma unroll
            for (int q = 0; q < 2; ++q) {
                const uint32_t cq = __shfl_sync(kFullMask, count, q);
                if (cq <= warp_max) continue;
                // a large group: the block's first one stays with it, further ones go to the grid-wide queue
                const uint32_t mq = __shfl_sync(kFullMask, M, q), oq = __shfl_sync(kFullMask, off, q), nq = __shfl_sync(kFullMask, nwords, q);
                if (lane == 0) {
                    const uint32_t nth = atomicAdd(&s.big_count, 1u);
                    if (nth == 0u) {
                        s.g_count[0] = cq; s.g_M[0] = mq; s.g_off[0] = oq; s.g_nwords[0] = nq;
                        s.local_g = g + (uint32_t)q * stride;
                    } else {
                        const uint32_t slot = atomicAdd(a.q_ctl + 4, 1u);
                        __threadfence();
                        *reinterpret_cast<volatile unsigned int*>(a.q_list + slot) = g + (uint32_t)q * stride + 1u;
                    }
                }
                if (lane == q) { count = 0u; nwords = 0u; }
            }
            if (!__any_sync(kFullMask, count != 0u)) continue;
            if (count == 0u) nwords = 0u;
            const uint32_t nw_incl = warp_incl_scan(nwords, lane);
            const uint32_t base = nw_incl - nwords;
            uint32_t* stage = s.u.wstage[warp];
            const uint32_t* b2[2]; uint32_t n2[2], c2[2], m2[2]; const float* v2[2];
#pragma unroll
            for (int q = 0; q < 2; ++q) {
                c2[q] = __shfl_sync(kFullMask, count, q); n2[q] = __shfl_sync(kFullMask, nwords, q);
                m2[q] = __shfl_sync(kFullMask, M, q); b2[q] = stage + __shfl_sync(kFullMask, base, q); v2[q] = s.val[0];
            }
            // both copies' loads in flight together
            {
                const uint32_t o0 = __shfl_sync(kFullMask, off, 0), o1 = __shfl_sync(kFullMask, off, 1);
                const uint32_t tot = n2[0] + n2[1];
                for (uint32_t i0 = 0; i0 < tot; i0 += 128u) {
                    uint32_t r[4];
#pragma unroll
                    for (int u = 0; u < 4; ++u) {
                        const uint32_t i = i0 + (uint32_t)u * 32u + (uint32_t)lane;
                        r[u] = i < n2[0] ? __ldg(sw0 + o0 + i) : (i < tot ? __ldg(sw0 + o1 + (i - n2[0])) : 0u);
                    }
#pragma unroll
                    for (int u = 0; u < 4; ++u) {
                        const uint32_t i = i0 + (uint32_t)u * 32u + (uint32_t)lane;
                        if (i < tot) stage[i] = r[u];          // (slot 1's blob follows slot 0's: base = n2[0])
                    }
                }
            }
            __syncwarp();
            // (one stream: a call always holds the whole group, so that mode 2 is decode_multi's own)
            if (c2[0] <= kDecWarpSide && c2[1] <= kDecWarpSide)
                decode_multi<MODE, false, 2, 4, true>(a, s, b2, n2, c2, m2, v2, g, nullptr, lane, 32, lane, warp, g + stride);
            else
                decode_multi<MODE, false, 2, 8, true>(a, s, b2, n2, c2, m2, v2, g, nullptr, lane, 32, lane, warp, g + stride);
            __syncwarp();
        }
    } else
    for (uint32_t g = blockIdx.x + warp * gridDim.x; g < a.G; g += kDecWarps * gridDim.x) {
        // lane w reads and checks stream w's directory entry
        uint32_t count = 0, M = 0, off = 0, nwords = 0;
        if (lane < (int)W && s.ok[lane])
            read_dir(a, reinterpret_cast<const uint32_t*>(a.stream[lane]), g, s.total_words[lane], &count, &M, &off, &nwords);
        if (!__any_sync(kFullMask, count != 0u)) continue;
        if (__any_sync(kFullMask, count > warp_max)) {
            // a large group: the first one the block finds is its own (directory entries kept in shared
            // memory), any further one goes to the grid-wide queue: reserve a slot, then fill it (g + 1: 0 = empty)
            uint32_t nth = 0;
            if (lane == 0) nth = atomicAdd(&s.big_count, 1u);
            nth = __shfl_sync(kFullMask, nth, 0);
            if (nth == 0u) {
                if (lane < (int)W) { s.g_count[lane] = count; s.g_M[lane] = M; s.g_off[lane] = off; s.g_nwords[lane] = nwords; }
                if (lane == 0) s.local_g = g;
            } else if (lane == 0) {
                const uint32_t slot = atomicAdd(a.q_ctl + 4, 1u);
                __threadfence();
                *reinterpret_cast<volatile unsigned int*>(a.q_list + slot) = g + 1u;
            }
            continue;
        }
        // copy the streams' blobs for this group into the warp's staging area
        if (count == 0u) nwords = 0u;
        const uint32_t nw_incl = warp_incl_scan(nwords, lane);
        const uint32_t base = nw_incl - nwords;
        uint32_t* stage = s.u.wstage[warp];
        for (uint32_t w = 0; w < W; ++w) {
            const uint32_t nw = __shfl_sync(kFullMask, nwords, w), b = __shfl_sync(kFullMask, base, w), o = __shfl_sync(kFullMask, off, w);
            const uint32_t* src = reinterpret_cast<const uint32_t*>(a.stream[w]) + o;
            for (uint32_t i = lane; i < nw; i += 32) stage[b + i] = __ldg(src + i);
        }
        __syncwarp();
        if (__any_sync(kFullMask, count > kDecWarpSide)) {
            // longer runs per lane: two streams at a time
            const bool fused = mode_fused(MODE) && W <= 2u;
            const int npass = (mode_fused(MODE) && !fused) ? 2 : 1;
            for (int pass = 0; pass < npass; ++pass)
            for (uint32_t w0 = 0; w0 < W; w0 += 2u) {
                const uint32_t w1 = w0 + 1u < W ? w0 + 1u : w0;
                const uint32_t* b2[2]; uint32_t n2[2], c2[2], m2[2]; const float* v2[2];
                c2[0] = __shfl_sync(kFullMask, count, w0); c2[1] = w0 + 1u < W ? __shfl_sync(kFullMask, count, w1) : 0u;
                b2[0] = stage + __shfl_sync(kFullMask, base, w0); b2[1] = stage + __shfl_sync(kFullMask, base, w1);
                n2[0] = __shfl_sync(kFullMask, nwords, w0); n2[1] = __shfl_sync(kFullMask, nwords, w1);
                m2[0] = __shfl_sync(kFullMask, M, w0); m2[1] = __shfl_sync(kFullMask, M, w1);
                v2[0] = s.val[w0]; v2[1] = s.val[w1];
                if (w0 + 1u < W) {
                    FSG_DECODE_MULTI(fused, false, 2, 8, false, a, s, b2, n2, c2, m2, v2, g, nullptr, lane, 32, lane, warp);
                } else {
                    const uint32_t* b1[1] = {b2[0]}; const uint32_t n1[1] = {n2[0]}, c1[1] = {c2[0]}, m1[1] = {m2[0]}; const float* v1[1] = {v2[0]};
                    FSG_DECODE_MULTI(fused, false, 1, 8, false, a, s, b1, n1, c1, m1, v1, g, nullptr, lane, 32, lane, warp);
                }
                __syncwarp();      // these streams' stores before the next streams' loads of the same keys
            }
        } else {
            if constexpr (mode_fused(MODE)) {
                if (W <= 4u) warp_fours<MODE>(a, s, stage, count, M, base, nwords, W, g, lane, warp);
                else {      // the update only after every stream's values are in
                    warp_fours<(MODE == 3 ? 4 : 0)>(a, s, stage, count, M, base, nwords, W, g, lane, warp);
                    warp_fours<(MODE == 3 ? 5 : 1)>(a, s, stage, count, M, base, nwords, W, g, lane, warp);
                }
            } else {
        // up to four streams at a time, parsed side by side and applied in stream order
        for (uint32_t w0 = 0; w0 < W; w0 += 4u) {
            const uint32_t ns = W - w0 < 4u ? W - w0 : 4u;
            const uint32_t* bl[4]; uint32_t nwv[4], cv[4], mv[4]; const float* vl[4];
#pragma unroll
            for (int i = 0; i < 4; ++i) {
                const uint32_t src = (uint32_t)i < ns ? w0 + i : w0;
                const uint32_t c = __shfl_sync(kFullMask, count, src), b = __shfl_sync(kFullMask, base, src);
                nwv[i] = __shfl_sync(kFullMask, nwords, src); mv[i] = __shfl_sync(kFullMask, M, src);
                cv[i] = (uint32_t)i < ns ? c : 0u;
                bl[i] = stage + b; vl[i] = s.val[src];
            }
            if (ns == 1u) {
                const uint32_t* b1[1] = {bl[0]}; const uint32_t n1[1] = {nwv[0]}, c1[1] = {cv[0]}, m1[1] = {mv[0]}; const float* v1[1] = {vl[0]};
                decode_multi<MODE, false, 1, 4>(a, s, b1, n1, c1, m1, v1, g, nullptr, lane, 32, lane, warp);
            } else if (ns == 2u) {
                const uint32_t* b2[2] = {bl[0], bl[1]}; const uint32_t n2[2] = {nwv[0], nwv[1]}, c2[2] = {cv[0], cv[1]}, m2[2] = {mv[0], mv[1]};
                const float* v2[2] = {vl[0], vl[1]};
                decode_multi<MODE, false, 2, 4>(a, s, b2, n2, c2, m2, v2, g, nullptr, lane, 32, lane, warp);
            } else {
                decode_multi<MODE, false, 4, 4>(a, s, bl, nwv, cv, mv, vl, g, nullptr, lane, 32, lane, warp);
            }
            __syncwarp();          // these streams' stores before the next streams' loads of the same keys
        }
            }
        }
    }
    __syncthreads();

    FSG_DEC_STAMP(T2);
    // ---- groups with many keys sit in a queue shared by all blocks, so that a block that found
    //      several of them does not hold the others up.  Slots are filled as the groups are found;
    //      a taker waits (bounded) for its slot, or leaves once every block is past its own groups
    //      and the slot lies beyond the last reservation.
    unsigned int* q_taken = a.q_ctl + 1, *q_done = a.q_ctl + 2, *q_exited = a.q_ctl + 3, *q_reserved = a.q_ctl + 4;
    if (tid == 0) { __threadfence(); atomicAdd(q_done, 1u); }
    const bool local_first = s.big_count > 0u;      // (written before the barrier above)
    for (uint32_t round = 0;; ++round) {
        const bool local = round == 0u && local_first;
        uint32_t g;
        if (local) {
            g = s.local_g;
        } else {
            if (tid == 0) {
                uint32_t got = 0xFFFFFFFFu;
                const uint32_t i = atomicAdd(q_taken, 1u);
                uint32_t spin = 0;
                for (;;) {
                    if (i < a.G) {
                        const uint32_t e = *reinterpret_cast<volatile unsigned int*>(a.q_list + i);
                        if (e != 0u) { got = e - 1u; *reinterpret_cast<volatile unsigned int*>(a.q_list + i) = 0u; break; }
                    }
                    if (*reinterpret_cast<volatile unsigned int*>(q_done) >= gridDim.x &&
                        i >= *reinterpret_cast<volatile unsigned int*>(q_reserved)) break;      // nothing will fill it
                    if (i >= a.G) break;
                    if (++spin > a.spin_limit) {         // the slot was reserved and never filled in time: the group it stands for is lost
                        dec_fail(a, 0u, 0u, kStTimeout);
                        break;
                    }
                    __nanosleep(100);
                }
                s.big[0] = got;
            }
            __syncthreads();
            g = s.big[0];
            if (g == 0xFFFFFFFFu) break;
        }
#ifdef FASTSGD_TRACE
        ++taken;
#endif
        const uint64_t lo64 = (uint64_t)g << a.group_log2;
        const uint64_t hi64 = lo64 + (1ull << a.group_log2);
        const uint32_t lo = (uint32_t)lo64, span = (uint32_t)((hi64 < a.n ? hi64 : a.n) - lo64);
        // The group's slice of dense_out is brought into shared memory by one bulk copy, updated there by
        // every stream in turn, and written back by one bulk copy (needs 16-byte alignment and size).
        // (packed state: the slice of g is only ever formed in shared memory, so the copies' alignment rules do not matter;
        //  the host admits no wider groups there)
        const bool use_tile = a.group_log2 <= 14u &&
                              (MODE == 3 || (((reinterpret_cast<uintptr_t>(a.dense) & 15u) == 0u) && ((span & 3u) == 0u)));
        // (modes 2 and 3: g is all zero by contract and is left so: the slice starts as zeros in shared memory and never leaves it)
        const bool load_tile = use_tile && !mode_fused(MODE);
        if (load_tile && tid == 0) {
            asm volatile("cp.async.bulk.wait_group.read 0;" ::: "memory");      // the last write-back has read the tile
            mbar_expect_tx(&s.tile_bar, span * 4u);
            bulk_load(s.u.tile, a.dense + lo, span * 4u, &s.tile_bar);
        }
        if (mode_fused(MODE) && use_tile)
            for (uint32_t i = tid; i < ((span + 3u) >> 2); i += kDecThreads)
                reinterpret_cast<float4*>(s.u.tile)[i] = make_float4(0.f, 0.f, 0.f, 0.f);
        if (!local && tid < (int)W) {
            uint32_t count = 0, M = 0, off = 0, nwords = 0;
            if (s.ok[tid])
                read_dir(a, reinterpret_cast<const uint32_t*>(a.stream[tid]), g, s.total_words[tid], &count, &M, &off, &nwords);
            s.g_count[tid] = count; s.g_M[tid] = M; s.g_off[tid] = off; s.g_nwords[tid] = nwords;
        }
        __syncthreads();
        // Model update with the group's slice of the aggregated gradient in shared memory: the streams need not be
        // parsed again -- the coordinates to update are the non-zeros of the slice.  Thread t looks at entries
        // t, t + 256, ..., eight at a time, so that the loads of their moments and parameters are in flight together
        // (neighbouring threads, neighbouring addresses).
        const bool scan_tile = MODE != 0 && use_tile;
        const bool parse = !(MODE == 1 && use_tile);
        // staging offsets; a blob that does not fit is parsed from global memory
        uint32_t used = 0;
        if (parse)
        for (uint32_t w = 0; w < W; ++w) {
            const uint32_t nw = s.g_count[w] ? s.g_nwords[w] : 0u;
            const bool fits = used + nw <= kBlockStageWords;
            if (tid == 0) { s.g_base[w] = used; s.g_valid[w] = fits ? 1u : 0u; }
            if (fits) {
                const uint32_t* src = reinterpret_cast<const uint32_t*>(a.stream[w]) + s.g_off[w];
                for (uint32_t i = tid; i < nw; i += kDecThreads) s.bstage[used + i] = __ldg(src + i);
                used += nw;
            }
        }
        __syncthreads();
        if (load_tile) {
            if (tid == 0) s.big[1] = mbar_wait(&s.tile_bar, tile_parity, a.try_limit) ? 1u : 0u;     // bounded wait, one thread
            __syncthreads();
            tile_parity ^= 1u;
            if (s.big[1] == 0u) {                                 // ran out: the group is skipped
                if (tid == 0) dec_fail(a, g, 0u, kStTimeout);
                __syncthreads();
                continue;
            }
        }
        // MODE 2 without the slice in shared memory: every stream aggregated into dense_out, then every stream again for the update
        const int npass = (mode_fused(MODE) && !use_tile) ? 2 : 1;
        if (parse)
        for (int pass = 0; pass < npass; ++pass)
        for (uint32_t w = 0; w < W; ++w) {
            const uint32_t c = s.g_count[w];
            const uint32_t* blob = s.g_valid[w] ? s.bstage + s.g_base[w]
                                                : reinterpret_cast<const uint32_t*>(a.stream[w]) + s.g_off[w];
            // short runs per thread: the leaner parser, two streams side by side where the next one qualifies too
            if (c <= 4u * (uint32_t)kDecThreads && w + 1u < W && s.g_count[w + 1u] <= 4u * (uint32_t)kDecThreads) {
                const uint32_t w2 = w + 1u;
                const uint32_t* blob2 = s.g_valid[w2] ? s.bstage + s.g_base[w2]
                                                      : reinterpret_cast<const uint32_t*>(a.stream[w2]) + s.g_off[w2];
                const uint32_t* b2[2] = {blob, blob2}; const uint32_t n2[2] = {s.g_nwords[w], s.g_nwords[w2]};
                const uint32_t c2[2] = {c, s.g_count[w2]}, m2[2] = {s.g_M[w], s.g_M[w2]};
                const float* v2[2] = {s.val[w], s.val[w2]};
                FSG_DECODE_MULTI_PASS(true, 2, 4, false, a, s, b2, n2, c2, m2, v2, g, use_tile ? s.u.tile : nullptr, tid, kDecThreads, lane, warp);
                ++w;
            } else if (c == 0u) {
                continue;
            } else if (c <= 4u * (uint32_t)kDecThreads) {
                const uint32_t* b1[1] = {blob}; const uint32_t n1[1] = {s.g_nwords[w]}, c1[1] = {c}, m1[1] = {s.g_M[w]};
                const float* v1[1] = {s.val[w]};
                FSG_DECODE_MULTI_PASS(true, 1, 4, false, a, s, b1, n1, c1, m1, v1, g, use_tile ? s.u.tile : nullptr, tid, kDecThreads, lane, warp);
            } else {
                if constexpr (mode_fused(MODE)) {
                    if (pass == 0) decode_long<0>(a, s, blob, s.g_nwords[w], g, c, s.g_M[w], s.val[w], use_tile ? s.u.tile : nullptr,
                                                  tid, kDecThreads, lane, warp);
                    else decode_long<1>(a, s, blob, s.g_nwords[w], g, c, s.g_M[w], s.val[w], use_tile ? s.u.tile : nullptr,
                                        tid, kDecThreads, lane, warp);
                } else {
                    decode_long<MODE>(a, s, blob, s.g_nwords[w], g, c, s.g_M[w], s.val[w], use_tile ? s.u.tile : nullptr,
                                      tid, kDecThreads, lane, warp);
                }
            }
            __syncthreads();       // these streams' updates before the next stream's
        }
        if (scan_tile) {
            for (uint32_t i0 = 0; i0 < span; i0 += 8u * (uint32_t)kDecThreads) {
                uint32_t kk[8]; float cur[8], vv[8], res[8];
#pragma unroll
                for (int u = 0; u < 8; ++u) {
                    const uint32_t idx = i0 + (uint32_t)u * (uint32_t)kDecThreads + (uint32_t)tid;
                    cur[u] = idx < span ? s.u.tile[idx] : 0.0f;
                    kk[u] = cur[u] != 0.0f ? lo + idx : 0xFFFFFFFFu;
                    vv[u] = 0.0f;
                }
                apply_run<1, 8, mode_packed(MODE)>(a, kk, cur, vv, res);
#pragma unroll
                for (int u = 0; u < 8; ++u)
                    if (kk[u] != 0xFFFFFFFFu) s.u.tile[i0 + (uint32_t)u * (uint32_t)kDecThreads + (uint32_t)tid] = res[u];
            }
            __syncthreads();
        }
        if (load_tile && tid == 0) {
            asm volatile("fence.proxy.async.shared::cta;" ::: "memory");          // the updates above, before the copy reads them
            asm volatile("cp.async.bulk.global.shared::cta.bulk_group [%0], [%1], %2;"
                         ::"l"(__cvta_generic_to_global(a.dense + lo)), "r"(smem_u32(s.u.tile)), "r"(span * 4u) : "memory");
            asm volatile("cp.async.bulk.commit_group;" ::: "memory");
        }
        __syncthreads();
    }
    if (tid == 0) asm volatile("cp.async.bulk.wait_group 0;" ::: "memory");        // write-backs complete before the block leaves
#ifdef FASTSGD_TRACE
    if (tid == 0 && blockIdx.x < 480u) {
        a.trace[8u * blockIdx.x + 0] = T0; a.trace[8u * blockIdx.x + 1] = T1; a.trace[8u * blockIdx.x + 2] = T2;
        a.trace[8u * blockIdx.x + 3] = read_globaltimer_dec(); a.trace[8u * blockIdx.x + 4] = taken;
    }
#endif
    // the last block to leave clears the counters for the next launch.  The slots were cleared as they were taken; a
    // slot whose taker gave up (status TIMEOUT) was filled afterwards with nobody to take it: cleared here, so that
    // the queue is back in its resting state whatever happened.
    if (tid == 0) {
        __threadfence();
        if (atomicAdd(q_exited, 1u) == gridDim.x - 1u) {
            if (*reinterpret_cast<volatile unsigned long long*>(a.status) != ~0ull) {
                const uint32_t reserved = *reinterpret_cast<volatile unsigned int*>(q_reserved);
                for (uint32_t i = 0; i < reserved && i < a.G; ++i) a.q_list[i] = 0u;
            }
            a.q_ctl[0] = 0u; *q_taken = 0u; *q_done = 0u; *q_reserved = 0u;
            __threadfence();
            *q_exited = 0u;
        }
    }
}

}  // namespace fsg
