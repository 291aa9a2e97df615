// Algorithm 2 as the paper prints it, on the GPU: ONE delta chain over all kept keys (preKey
// starts at 0), ONE M = max(1, bitlen(maxDelta)), and BK = flag || delta for each key in turn,
// most significant bit first.  (The product stream of compress.cuh splits the chain into groups
// and stores flags and deltas as two planes; this writer exists to state the paper's own format
// and its size per key.)
//
// Output buffer: 16-byte header {u32 M, u32 l, u64 number of bits} | index: one u64 per block of
// 2048 keys, the bit offset of that block's first key in BK | BK, zero-padded to a multiple of
// 4 bytes.  Four small launches on the caller's stream: largest delta; bits per block; scan of
// the blocks (one block); packing.  A block packs its 2048 keys in shared memory and stores whole
// words; only the first and the last word of its range, which it may share with a neighbour, are
// ORed into memory (the scan launch has zeroed them).
#pragma once

#include "common.cuh"
#include "bits.cuh"

namespace fsg {

constexpr int      kBkThreads     = 256;
constexpr int      kBkPerThread   = 8;
constexpr uint32_t kBkBlockKeys   = kBkThreads * kBkPerThread;              // 2048
constexpr uint32_t kBkBlockWords  = (kBkBlockKeys * (5u + 32u) + 31u) / 32u + 2u;   // widest block + the shift of its first word

struct BkArgs {
    const uint32_t*     keys;       // ascending (equal keys allowed only in the sense of Algorithm 2: a delta of 0)
    uint64_t            d;
    uint32_t*           header;     // out: {M (the largest delta until the scan launch), l, bits lo, bits hi}
    unsigned long long* index;      // out + 16: per block, first its bits, after the scan launch its bit offset
    uint32_t*           bk;         // out + 16 + 8 * blocks
    uint32_t            l;
    uint32_t            blocks;
};

__device__ __forceinline__ uint32_t bk_delta(const BkArgs& a, uint64_t j) {
    return __ldg(a.keys + j) - (j ? __ldg(a.keys + j - 1) : 0u);
}

// bits of one key: the flag's l bits plus the width its flag selects (Sec. 3.3: level f holds ceil((f+1) M / 2^l) bits)
__device__ __forceinline__ uint32_t bk_flag(uint32_t delta, uint32_t M, uint32_t l) {
    const uint32_t need = 32u - (uint32_t)__clz((int)delta);      // bitlen, 0 for 0
    return need ? ((need - 1u) << l) / M : 0u;
}
__device__ __forceinline__ uint32_t bk_width(uint32_t flag, uint32_t M, uint32_t l) {
    return ((flag + 1u) * M + (1u << l) - 1u) >> l;
}

__global__ void __launch_bounds__(kBkThreads) k_bk_maxdelta(const BkArgs a) {
    uint32_t mx = 0;
    for (uint64_t j = (uint64_t)blockIdx.x * kBkThreads + threadIdx.x; j < a.d; j += (uint64_t)gridDim.x * kBkThreads)
        mx = max(mx, bk_delta(a, j));
    mx = __reduce_max_sync(kFullMask, mx);
    if ((threadIdx.x & 31) == 0 && mx) atomicMax(a.header, mx);
}

// Per-thread sizes of its 8 consecutive keys and the block-wide exclusive scan of the threads' sums.
__device__ __forceinline__ uint32_t bk_block_scan(uint32_t v, uint32_t* total, uint32_t* s_scan, int lane, int warp) {
    const uint32_t incl = warp_incl_scan(v, lane);
    if (lane == 31) s_scan[warp] = incl;
    __syncthreads();
    uint32_t before = 0, all = 0;
#pragma unroll
    for (int w = 0; w < kBkThreads / 32; ++w) {
        const uint32_t t = s_scan[w];
        if (w < warp) before += t;
        all += t;
    }
    *total = all;
    return before + incl - v;
}

__global__ void __launch_bounds__(kBkThreads) k_bk_sizes(const BkArgs a) {
    __shared__ uint32_t s_scan[kBkThreads / 32];
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const uint32_t maxd = a.header[0];
    const uint32_t M = maxd ? 32u - (uint32_t)__clz((int)maxd) : 1u;
    const uint64_t j0 = (uint64_t)blockIdx.x * kBkBlockKeys + (uint64_t)tid * kBkPerThread;
    uint32_t bits = 0;
#pragma unroll
    for (int k = 0; k < kBkPerThread; ++k)
        if (j0 + k < a.d) bits += a.l + bk_width(bk_flag(bk_delta(a, j0 + k), M, a.l), M, a.l);
    uint32_t total;
    bk_block_scan(bits, &total, s_scan, lane, warp);
    if (tid == 0) a.index[blockIdx.x] = total;
}

// One block: exclusive scan of the blocks' bits in place, the header, and zeroes in every word where two blocks meet.
__global__ void __launch_bounds__(kBkThreads) k_bk_scan(const BkArgs a) {
    __shared__ unsigned long long s_tot[kBkThreads / 32];
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    unsigned long long running = 0ull;
    for (uint32_t base = 0; base < a.blocks; base += kBkThreads) {
        const uint32_t b = base + tid;
        const unsigned long long v = b < a.blocks ? a.index[b] : 0ull;
        unsigned long long incl = v;
#pragma unroll
        for (int o = 1; o < 32; o <<= 1) {
            const unsigned long long t = __shfl_up_sync(kFullMask, incl, o);
            if (lane >= o) incl += t;
        }
        if (lane == 31) s_tot[warp] = incl;
        __syncthreads();
        unsigned long long before = running, all = 0ull;
#pragma unroll
        for (int w = 0; w < kBkThreads / 32; ++w) {
            const unsigned long long t = s_tot[w];
            if (w < warp) before += t;
            all += t;
        }
        const unsigned long long excl = before + incl - v;
        if (b < a.blocks) {
            a.index[b] = excl;
            a.bk[excl >> 5] = 0u;                             // the word this block starts in
            a.bk[(excl + v) >> 5] = 0u;                       // ... and the one it ends in (the padding word after the last block)
        }
        running += all;
        __syncthreads();
    }
    if (tid == 0) {
        const uint32_t maxd = a.header[0];
        a.header[0] = maxd ? 32u - (uint32_t)__clz((int)maxd) : 1u;
        a.header[1] = a.l;
        a.header[2] = (uint32_t)running;
        a.header[3] = (uint32_t)(running >> 32);
        if (a.blocks == 0u) a.bk[0] = 0u;
    }
}

__global__ void __launch_bounds__(kBkThreads) k_bk_pack(const BkArgs a) {
    __shared__ uint32_t s_scan[kBkThreads / 32];
    __shared__ uint32_t s_words[kBkBlockWords];
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const uint32_t M = a.header[0];
    const unsigned long long boff = a.index[blockIdx.x];
    const uint64_t j0 = (uint64_t)blockIdx.x * kBkBlockKeys + (uint64_t)tid * kBkPerThread;
    uint32_t dl[kBkPerThread], fl[kBkPerThread], wd[kBkPerThread];
    uint32_t bits = 0;
#pragma unroll
    for (int k = 0; k < kBkPerThread; ++k) {
        dl[k] = 0u; fl[k] = 0u; wd[k] = 0u;
        if (j0 + k < a.d) {
            dl[k] = bk_delta(a, j0 + k);
            fl[k] = bk_flag(dl[k], M, a.l);
            wd[k] = bk_width(fl[k], M, a.l);
            bits += a.l + wd[k];
        }
    }
    for (uint32_t i = tid; i < kBkBlockWords; i += kBkThreads) s_words[i] = 0u;
    uint32_t total;
    uint32_t pos = (uint32_t)(boff & 31ull) + bk_block_scan(bits, &total, s_scan, lane, warp);   // (the barrier inside also covers the zeroing)
#pragma unroll
    for (int k = 0; k < kBkPerThread; ++k) {
        if (j0 + k < a.d) {
            put_bits_smem(s_words, pos, fl[k], a.l);
            put_bits_smem(s_words, pos + a.l, dl[k], wd[k]);
            pos += a.l + wd[k];
        }
    }
    __syncthreads();
    const uint32_t first = (uint32_t)(boff >> 5);            // (BK of fewer than 2^37 bits)
    const uint32_t nw = ((uint32_t)(boff & 31ull) + total + 31u) >> 5;
    // a word is shared with a neighbouring block iff the block's range starts or ends inside it
    const bool shared_first = (boff & 31ull) != 0ull, shared_last = ((boff + total) & 31ull) != 0ull;
    for (uint32_t i = tid; i < nw; i += kBkThreads) {
        const uint32_t w = bswap32(s_words[i]);
        if ((i == 0u && shared_first) || (i + 1u == nw && shared_last)) { if (w) atomicOr(a.bk + first + i, w); }
        else a.bk[first + i] = w;
    }
}

}  // namespace fsg
