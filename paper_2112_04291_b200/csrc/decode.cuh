// Decoder (decoder phases 1-4) and aggregation, one warp per group.
//
// Phase 1: the length flags give every delta's width; an exclusive scan of the widths gives
// its bit offset.  Phase 2: an inclusive scan of the deltas, started at g*T, gives the keys
// back.  Phases 3-4: code L -> sum / b^L (the boundary B_L rounded to fp32), signed.  The
// aggregation adds the value into dense_out[key].  Keys are unique within a stream and calls
// are ordered by the CUDA stream, so the read-modify-write needs no atomics and the result
// does not depend on the launch shape.
#pragma once

#include "common.cuh"
#include "encode.cuh"

namespace fsg {

constexpr int kDecThreads = 256;

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

__global__ void __launch_bounds__(kDecThreads)
k_decode_accumulate(const DecArgs a, const __grid_constant__ PowTable pw) {
    __shared__ float s_val[132];
    __shared__ int s_status;
    __shared__ unsigned long long s_total;
    __shared__ double s_sum;
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const uint32_t* sw = reinterpret_cast<const uint32_t*>(a.stream);

    if (tid == 0) {
        uint32_t h[16];
#pragma unroll
        for (int i = 0; i < 16; ++i) h[i] = __ldg(sw + i);
        uint64_t total = 0; double S = 0.0;
        const int st = check_header(a, h, &total, &S);
        s_status = st; s_total = total; s_sum = S;
        if (st != kStOk && blockIdx.x == 0) dec_fail(a, 0u, 0u, st);
    }
    __syncthreads();
    if (s_status != kStOk) return;
    // phases 3-4 as a table: value[L] = (float)(sum / b^L)
    if (tid <= (int)a.tau) s_val[tid] = __double2float_rn(__ddiv_rn(s_sum, pw.P[tid]));
    __syncthreads();

    const uint32_t total_words = (uint32_t)(s_total >> 2);
    const uint32_t fixed_words = (kHeaderBytes + 8u * a.G) >> 2;
    const uint32_t T = 1u << a.group_log2;
    const uint32_t levels_m1 = (1u << a.l) - 1u;
    const uint32_t* dir = sw + (kHeaderBytes >> 2);

    const uint32_t warps_total = gridDim.x * (kDecThreads / 32);
    for (uint32_t g = blockIdx.x * (kDecThreads / 32) + warp; g < a.G; g += warps_total) {
        const uint32_t e0 = __ldg(dir + 2 * g), off = __ldg(dir + 2 * g + 1);
        const uint32_t next_off = (g + 1 < a.G) ? __ldg(dir + 2 * g + 3) : total_words;
        const uint32_t count = e0 & 0xFFFFFFu, M = e0 >> 24;
        const uint64_t lo64 = (uint64_t)g << a.group_log2;
        const uint32_t lo = (uint32_t)lo64;
        const uint32_t hi = (uint32_t)min((uint64_t)a.n, lo64 + T);
        if ((g == 0 && off != fixed_words) || next_off < off || next_off > total_words || off < fixed_words) {
            if (lane == 0) dec_fail(a, g, 0u, kStBadDirectory);
            continue;
        }
        if (count == 0) {
            if ((e0 != 0u || next_off != off) && lane == 0) dec_fail(a, g, 0u, kStBadDirectory);
            continue;
        }
        const uint32_t nwords = next_off - off;
        const uint64_t avail_bits = 32ull * nwords;
        const uint32_t flag_pos0 = 8u * count;
        const uint64_t delta_pos0_64 = (uint64_t)flag_pos0 + (uint64_t)a.l * count;
        if (count > hi - lo || M < 1u || M > a.group_log2 || delta_pos0_64 > avail_bits) {
            if (lane == 0) dec_fail(a, g, 0u, kStBadDirectory);
            continue;
        }
        const uint32_t delta_pos0 = (uint32_t)delta_pos0_64;
        const uint32_t* blob = sw + off;

        // phase 1a: the flags fix the blob's length; it must be the directory's
        uint32_t wsum = 0;
        for (uint32_t j = lane; j < count; j += 32) {
            const uint32_t f = get_bits_be(blob, nwords, flag_pos0 + a.l * j, a.l);
            wsum += ((f + 1u) * M + levels_m1) >> a.l;
        }
        wsum = __reduce_add_sync(kFullMask, wsum);
        if ((((uint64_t)delta_pos0 + wsum + 31ull) >> 5) != nwords) {
            if (lane == 0) dec_fail(a, g, 0u, kStBadDirectory);
            continue;
        }

        uint32_t carry_pos = delta_pos0, carry_key = lo;
        for (uint32_t j0 = 0; j0 < count; j0 += 32) {
            const uint32_t j = j0 + lane;
            const bool act = j < count;
            uint32_t w = 0, code = 0;
            if (act) {
                const uint32_t f = get_bits_be(blob, nwords, flag_pos0 + a.l * j, a.l);
                w = ((f + 1u) * M + levels_m1) >> a.l;
                code = (__ldg(blob + (j >> 2)) >> (8u * (j & 3u))) & 0xFFu;
            }
            const uint32_t w_incl = warp_incl_scan(w, lane);
            const uint32_t delta = act ? get_bits_be(blob, nwords, carry_pos + (w_incl - w), w) : 0u;
            const uint32_t d_incl = warp_incl_scan(delta, lane);
            const uint32_t key = carry_key + d_incl;
            const uint32_t L = (code & 0x7Fu) + 1u;
            const bool bad_key = act && ((j > 0 && delta == 0u) || key >= hi);
            const bool bad_code = act && L > a.tau;
            const uint32_t bad = __ballot_sync(kFullMask, bad_key || bad_code);
            if (bad) {
                const int first = __ffs(bad) - 1;
                if (lane == first) dec_fail(a, g, j, bad_key ? kStBadKey : kStBadCode);
                break;
            }
            if (act) {
                const float vhat = (code & 0x80u) ? -s_val[L] : s_val[L];
                a.dense[key] = __fadd_rn(a.dense[key], vhat);
            }
            carry_pos += __shfl_sync(kFullMask, w_incl, 31);
            carry_key += __shfl_sync(kFullMask, d_incl, 31);
        }
    }
}

}  // namespace fsg
