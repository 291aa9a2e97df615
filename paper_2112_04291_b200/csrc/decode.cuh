// Decoder (decoder phases 1-4) and aggregation.
//
// Phase 1: the length flags give every delta's width; an exclusive scan of the widths gives
// its bit offset.  Phase 2: an inclusive scan of the deltas, started at g*T, gives the keys
// back.  Phases 3-4: code L -> sum / b^L (the boundary B_L rounded to fp32), signed.  The
// aggregation adds the value into dense_out[key].  Keys are unique within a stream and calls
// are ordered by the CUDA stream, so the read-modify-write needs no atomics and the result
// does not depend on the launch shape.
//
// Work split: a group with few keys is decoded by one warp, a group with many keys by the
// whole block; either way a thread owns a run of consecutive keys, so that the scans are one
// shuffle scan (plus one shared-memory step for the block) per group instead of one per 32 keys,
// and a group is validated in full before any of it is applied.
#pragma once

#include "common.cuh"
#include "encode.cuh"

namespace fsg {

constexpr int      kDecThreads   = 256;
constexpr int      kDecWarps     = kDecThreads / 32;
constexpr uint32_t kDecWarpMax   = 128;     // groups with more keys go to the whole block
constexpr int      kDecListMax   = 512;     // groups one block may own

struct DecArgs {
    const uint8_t*      stream;
    uint64_t            bytes;
    uint64_t            n;
    float*              dense;
    unsigned long long* status;     // sticky minimum of (group << 32 | key index << 8 | status)
    double              base;
    uint32_t            G;
    uint32_t            tau;
    uint32_t            l;
    uint32_t            group_log2;
};

__device__ __forceinline__ void dec_fail(const DecArgs& a, uint32_t g, uint32_t j, int st) {
    atomicMin(a.status, ((unsigned long long)g << 32) | ((unsigned long long)(j & 0xFFFFFFu) << 8) | (unsigned)st);
}

__device__ __forceinline__ int check_header(const DecArgs& a, const uint32_t* w, uint64_t* total_out, double* sum_out) {
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
    if (total > a.bytes || total < fixed || (total & 3ull)) return kStTruncated;
    *total_out = total;
    *sum_out = __longlong_as_double((long long)((unsigned long long)w[10] | ((unsigned long long)w[11] << 32)));
    return kStOk;
}

struct DecShared {
    float              val[132];
    uint32_t           scan[kDecWarps];
    uint32_t           big[kDecListMax];
    unsigned long long first_bad;     // min over threads of (key index << 8 | status), block path
    uint32_t           big_count;
    int                status;
    unsigned long long total;
    double             sum;
};

// exclusive scan of one value per thread over the warp (BLOCK = false) or the block; also returns the total
template <bool BLOCK>
__device__ __forceinline__ uint32_t excl_scan(uint32_t v, uint32_t* total, DecShared& s, int lane, int warp) {
    const uint32_t incl = warp_incl_scan(v, lane);
    if (!BLOCK) {
        *total = __shfl_sync(kFullMask, incl, 31);
        return incl - v;
    }
    __syncthreads();                       // s.scan may still be read from the previous scan
    if (lane == 31) s.scan[warp] = incl;
    __syncthreads();
    uint32_t before = 0, all = 0;
#pragma unroll
    for (int w = 0; w < kDecWarps; ++w) {
        const uint32_t t = s.scan[w];
        if (w < warp) before += t;
        all += t;
    }
    *total = all;
    return before + incl - v;
}

// One group, decoded by a warp (BLOCK = false, `t` = lane, `nthreads` = 32) or by the block.
template <bool BLOCK>
__device__ __forceinline__ void decode_group(const DecArgs& a, DecShared& s, const uint32_t* __restrict__ sw,
                                             uint32_t g, uint32_t total_words, uint32_t fixed_words,
                                             int t, int nthreads, int lane, int warp) {
    const uint32_t* dir = sw + (kHeaderBytes >> 2);
    const uint32_t e0 = __ldg(dir + 2 * g), off = __ldg(dir + 2 * g + 1);
    const uint32_t next_off = (g + 1 < a.G) ? __ldg(dir + 2 * g + 3) : total_words;
    const uint32_t count = e0 & 0xFFFFFFu, M = e0 >> 24;
    const uint64_t lo64 = (uint64_t)g << a.group_log2;
    const uint32_t lo = (uint32_t)lo64;
    const uint64_t hi64 = lo64 + (1ull << a.group_log2);
    const uint32_t hi = (uint32_t)(hi64 < a.n ? hi64 : a.n);
    const bool lead = (t == 0);
    if ((g == 0 && off != fixed_words) || next_off < off || next_off > total_words || off < fixed_words) {
        if (lead) dec_fail(a, g, 0u, kStBadDirectory);
        return;
    }
    if (count == 0) {
        if ((e0 != 0u || next_off != off) && lead) dec_fail(a, g, 0u, kStBadDirectory);
        return;
    }
    const uint32_t nwords = next_off - off;
    const uint64_t avail_bits = 32ull * nwords;
    const uint32_t flag_pos0 = 8u * count;
    const uint64_t delta_pos0_64 = (uint64_t)flag_pos0 + (uint64_t)a.l * count;
    if (count > hi - lo || M < 1u || M > a.group_log2 || delta_pos0_64 > avail_bits) {
        if (lead) dec_fail(a, g, 0u, kStBadDirectory);
        return;
    }
    const uint32_t delta_pos0 = (uint32_t)delta_pos0_64;
    const uint32_t* blob = sw + off;
    const uint32_t levels_m1 = (1u << a.l) - 1u;

    // this thread's run of consecutive keys [jb, je)
    const uint32_t K = (count + nthreads - 1) / nthreads;
    const uint32_t jb = min(count, (uint32_t)t * K), je = min(count, jb + K);

    // phase 1: widths from the flags; their sum fixes the blob's length, which must be the directory's
    uint32_t wsum = 0;
    for (uint32_t j = jb; j < je; ++j) {
        const uint32_t f = get_bits_be(blob, nwords, flag_pos0 + a.l * j, a.l);
        wsum += ((f + 1u) * M + levels_m1) >> a.l;
    }
    uint32_t wtotal;
    const uint32_t pos0 = delta_pos0 + excl_scan<BLOCK>(wsum, &wtotal, s, lane, warp);
    if ((((uint64_t)delta_pos0 + wtotal + 31ull) >> 5) != nwords) {
        if (lead) dec_fail(a, g, 0u, kStBadDirectory);
        return;
    }

    // phase 2: sum of this thread's deltas, then the key before its first one
    uint32_t dsum = 0;
    {
        uint32_t pos = pos0;
        for (uint32_t j = jb; j < je; ++j) {
            const uint32_t f = get_bits_be(blob, nwords, flag_pos0 + a.l * j, a.l);
            const uint32_t w = ((f + 1u) * M + levels_m1) >> a.l;
            dsum = min(dsum + get_bits_be(blob, nwords, pos, w), 1u << 21);   // saturates only when already invalid
            pos += w;
        }
    }
    uint32_t dtotal;
    const uint32_t key0 = lo + excl_scan<BLOCK>(dsum, &dtotal, s, lane, warp);

    // validation of the whole group before anything is applied: first key index that repeats,
    // leaves the group, or carries a code beyond tau
    unsigned long long bad = ~0ull;
    {
        uint32_t pos = pos0, key = key0;
        for (uint32_t j = jb; j < je; ++j) {
            const uint32_t f = get_bits_be(blob, nwords, flag_pos0 + a.l * j, a.l);
            const uint32_t w = ((f + 1u) * M + levels_m1) >> a.l;
            const uint32_t delta = get_bits_be(blob, nwords, pos, w);
            pos += w;
            key += delta;
            const uint32_t code = (__ldg(blob + (j >> 2)) >> (8u * (j & 3u))) & 0xFFu;
            if ((j > 0 && delta == 0u) || key >= hi) { bad = ((unsigned long long)j << 8) | (unsigned)kStBadKey; break; }
            if ((code & 0x7Fu) + 1u > a.tau) { bad = ((unsigned long long)j << 8) | (unsigned)kStBadCode; break; }
        }
    }
    if (BLOCK) {
        __syncthreads();
        if (t == 0) s.first_bad = ~0ull;
        __syncthreads();
        if (bad != ~0ull) atomicMin(&s.first_bad, bad);
        __syncthreads();
        bad = s.first_bad;
    } else {
        const uint32_t blo = __reduce_min_sync(kFullMask, (uint32_t)(bad < 0xFFFFFFFFull ? bad : 0xFFFFFFFFull));
        bad = blo == 0xFFFFFFFFu ? ~0ull : (unsigned long long)blo;
    }
    if (bad != ~0ull) {
        if (lead) dec_fail(a, g, (uint32_t)(bad >> 8), (int)(bad & 0xFFull));
        return;
    }

    // phases 3-4 and the aggregation, four keys at a time (distinct keys: no aliasing)
    {
        uint32_t pos = pos0, key = key0;
        for (uint32_t j = jb; j < je; j += 4) {
            uint32_t kk[4]; float vv[4], dd[4];
#pragma unroll
            for (int i = 0; i < 4; ++i) {
                kk[i] = 0xFFFFFFFFu; vv[i] = 0.f;
                if (j + i < je) {
                    const uint32_t f = get_bits_be(blob, nwords, flag_pos0 + a.l * (j + i), a.l);
                    const uint32_t w = ((f + 1u) * M + levels_m1) >> a.l;
                    key += get_bits_be(blob, nwords, pos, w);
                    pos += w;
                    const uint32_t code = (__ldg(blob + ((j + i) >> 2)) >> (8u * ((j + i) & 3u))) & 0xFFu;
                    const float mag = s.val[(code & 0x7Fu) + 1u];
                    kk[i] = key; vv[i] = (code & 0x80u) ? -mag : mag;
                }
            }
#pragma unroll
            for (int i = 0; i < 4; ++i) dd[i] = kk[i] != 0xFFFFFFFFu ? a.dense[kk[i]] : 0.f;
#pragma unroll
            for (int i = 0; i < 4; ++i) if (kk[i] != 0xFFFFFFFFu) a.dense[kk[i]] = __fadd_rn(dd[i], vv[i]);
        }
    }
}

__global__ void __launch_bounds__(kDecThreads)
k_decode_accumulate(const DecArgs a, const __grid_constant__ PowTable pw) {
    __shared__ DecShared s;
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const uint32_t* sw = reinterpret_cast<const uint32_t*>(a.stream);

    if (tid == 0) {
        uint32_t h[16];
#pragma unroll
        for (int i = 0; i < 16; ++i) h[i] = __ldg(sw + i);
        uint64_t total = 0; double S = 0.0;
        const int st = check_header(a, h, &total, &S);
        s.status = st; s.total = total; s.sum = S; s.big_count = 0u;
        if (st != kStOk && blockIdx.x == 0) dec_fail(a, 0u, 0u, st);
    }
    __syncthreads();
    if (s.status != kStOk) return;
    // phases 3-4 as a table: value[L] = (float)(sum / b^L)
    if (tid <= (int)a.tau) s.val[tid] = __double2float_rn(__ddiv_rn(s.sum, pw.P[tid]));
    __syncthreads();

    const uint32_t total_words = (uint32_t)(s.total >> 2);
    const uint32_t fixed_words = (kHeaderBytes + 8u * a.G) >> 2;
    const uint32_t* dir = sw + (kHeaderBytes >> 2);

    // this block owns groups blockIdx.x, blockIdx.x + gridDim.x, ...; warp w takes every 8th of them
    uint32_t i = warp;
    for (uint32_t g = blockIdx.x + warp * gridDim.x; g < a.G; g += kDecWarps * gridDim.x, i += kDecWarps) {
        const uint32_t count = __ldg(dir + 2 * g) & 0xFFFFFFu;
        if (count > kDecWarpMax) {
            if (lane == 0) { const uint32_t slot = atomicAdd(&s.big_count, 1u); if (slot < kDecListMax) s.big[slot] = g; }
            continue;
        }
        decode_group<false>(a, s, sw, g, total_words, fixed_words, lane, 32, lane, warp);
    }
    __syncthreads();
    const uint32_t nbig = min(s.big_count, (uint32_t)kDecListMax);
    for (uint32_t b = 0; b < nbig; ++b)
        decode_group<true>(a, s, sw, s.big[b], total_words, fixed_words, tid, kDecThreads, lane, warp);
}

}  // namespace fsg
