// Second pass of the encoder: threshold filter, logarithm quantisation (Algorithm 1), and the
// key encoder (Algorithm 2) per group of T = 2^14 consecutive indices, in one kernel.
//
// One thread block takes one group (ticketed, so that a block's predecessors are always
// running or done): loads its 64 KiB tile with 128-bit loads, compacts the kept entries in
// index order (ballot-free packed warp scan), quantises them against the boundary table,
// forms the deltas, picks M and the length flags, scans the widths, packs codes | flags |
// deltas into shared memory, obtains its blob's offset in the stream by decoupled look-back
// over (count, words) descriptors, and copies the blob out with coalesced word stores.
#pragma once

#include "common.cuh"
#include "sum.cuh"

namespace fsg {

constexpr int      kEncThreads   = 512;
constexpr int      kEncWarps     = kEncThreads / 32;
constexpr int      kGroupLog2    = 14;
constexpr uint32_t kGroup        = 1u << kGroupLog2;
// widest blob: every entry kept, l = 5, M = 14
constexpr uint32_t kBlobWordsMax = (kGroup * (8u + 5u + (uint32_t)kGroupLog2) + 31u) / 32u;
constexpr uint32_t kLookbackSpinLimit = 4u << 20;   // polls of one descriptor window before giving up

struct EncSmem {
    float    thr[132];
    uint32_t wtab[32];          // width of level f
    uint32_t ftab[24];          // level of a delta with a given bit length
    uint32_t warp_tot[kEncWarps];
    uint32_t scan_tot[kEncWarps];
    uint32_t ticket;
    uint32_t max_delta;
    uint32_t excl_count;
    uint32_t excl_words;
    uint32_t poisoned;
    uint32_t pad[3];
    uint32_t blob[kBlobWordsMax];
    uint16_t keys[kGroup];
    uint8_t  codes[kGroup];
};

struct EncArgs {
    const float*        grad;
    uint64_t            n;
    uint8_t*            out;
    uint64_t            out_bytes;
    Control*            ctl;
    const float*        thr;
    unsigned long long* desc;
    double              base;
    uint32_t            G;
    uint32_t            tau;
    uint32_t            l;
};

// OR `nb` bits (value < 2^nb, nb <= 32) into a zeroed most-significant-bit-first sequence held
// as big-endian-valued 32-bit words in shared memory
__device__ __forceinline__ void put_bits_smem(uint32_t* blob, uint32_t pos, uint32_t value, uint32_t nb) {
    if (nb == 0) return;
    const uint32_t wi = pos >> 5, sh = pos & 31u;
    if (sh + nb <= 32u) {
        atomicOr(&blob[wi], value << (32u - sh - nb));
    } else {
        const uint32_t spill = sh + nb - 32u;          // bits that go to the next word
        atomicOr(&blob[wi], value >> spill);
        atomicOr(&blob[wi + 1], value << (32u - spill));
    }
}

__device__ __forceinline__ uint32_t warp_incl_scan(uint32_t v, int lane) {
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) {
        uint32_t t = __shfl_up_sync(kFullMask, v, o);
        if (lane >= o) v += t;
    }
    return v;
}

__global__ void __launch_bounds__(kEncThreads, 2)
k_encode(const EncArgs a) {
    extern __shared__ __align__(16) unsigned char smem_raw[];
    EncSmem& s = *reinterpret_cast<EncSmem*>(smem_raw);
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;

    if (tid == 0) {
        s.ticket = atomicAdd(&a.ctl->ticket, 1u);
        s.max_delta = 0u;
        s.poisoned = 0u;
    }
    if (tid <= (int)a.tau) s.thr[tid] = a.thr[tid];
    const uint32_t skip = a.ctl->skip;
    __syncthreads();
    const uint32_t g = s.ticket;
    if (g >= a.G) return;
    const uint64_t tile0 = (uint64_t)g << kGroupLog2;
    const float thr_e = s.thr[a.tau];                    // tau_e as an fp32 compare

    // ---- threshold filter on the tile: kept mask, bit 4r+c <-> entry warp*1024 + r*128 + lane*4 + c
    uint32_t m = 0;
    if (!skip) {
        const uint64_t base = tile0 + (uint64_t)warp * 1024u + (uint64_t)lane * 4u;
        float4 v[8];
        if (tile0 + kGroup <= a.n) {
#pragma unroll
            for (int r = 0; r < 8; ++r) v[r] = __ldg(reinterpret_cast<const float4*>(a.grad + base + r * 128));
        } else {
#pragma unroll
            for (int r = 0; r < 8; ++r) v[r] = load4_guarded(a.grad, base + r * 128, a.n);
        }
#pragma unroll
        for (int r = 0; r < 8; ++r) {
            m |= (fabsf(v[r].x) >= thr_e ? 1u : 0u) << (4 * r);
            m |= (fabsf(v[r].y) >= thr_e ? 1u : 0u) << (4 * r + 1);
            m |= (fabsf(v[r].z) >= thr_e ? 1u : 0u) << (4 * r + 2);
            m |= (fabsf(v[r].w) >= thr_e ? 1u : 0u) << (4 * r + 3);
        }
    }

    // ---- stream compaction in index order.  Per row the lanes' counts (<= 4 each, <= 128 per
    // row) are scanned four rows at a time, one byte per row.
    uint32_t ex0 = 0, ex1 = 0, tot0 = 0, tot1 = 0, warp_total = 0;
    const bool warp_any = __any_sync(kFullMask, m != 0u);
    if (warp_any) {
        uint32_t c0 = 0, c1 = 0;
#pragma unroll
        for (int r = 0; r < 4; ++r) {
            c0 |= (uint32_t)__popc((m >> (4 * r)) & 0xFu) << (8 * r);
            c1 |= (uint32_t)__popc((m >> (4 * (r + 4))) & 0xFu) << (8 * r);
        }
        const uint32_t i0 = warp_incl_scan(c0, lane), i1 = warp_incl_scan(c1, lane);
        ex0 = i0 - c0; ex1 = i1 - c1;
        tot0 = __shfl_sync(kFullMask, i0, 31); tot1 = __shfl_sync(kFullMask, i1, 31);
#pragma unroll
        for (int r = 0; r < 4; ++r) warp_total += ((tot0 >> (8 * r)) & 0xFFu) + ((tot1 >> (8 * r)) & 0xFFu);
    }
    if (lane == 0) s.warp_tot[warp] = warp_total;
    __syncthreads();
    uint32_t warp_base = 0, count = 0;
#pragma unroll
    for (int w = 0; w < kEncWarps; ++w) {
        const uint32_t t = s.warp_tot[w];
        if (w < warp) warp_base += t;
        count += t;
    }
    if (m != 0u) {
        uint32_t row_base = warp_base;
#pragma unroll
        for (int r = 0; r < 8; ++r) {
            const uint32_t tot = r < 4 ? (tot0 >> (8 * r)) & 0xFFu : (tot1 >> (8 * (r - 4))) & 0xFFu;
            const uint32_t ex  = r < 4 ? (ex0 >> (8 * r)) & 0xFFu : (ex1 >> (8 * (r - 4))) & 0xFFu;
            const uint32_t mr = (m >> (4 * r)) & 0xFu;
            uint32_t pos = row_base + ex;
#pragma unroll
            for (int c = 0; c < 4; ++c) {
                if (mr & (1u << c)) {
                    s.keys[pos] = (uint16_t)(warp * 1024 + r * 128 + lane * 4 + c);
                    ++pos;
                }
            }
            row_base += tot;
        }
    }
    __syncthreads();

    // ---- logarithm quantisation of the kept entries and the delta keys
    {
        uint32_t local_max = 0;
        for (uint32_t j = tid; j < count; j += kEncThreads) {
            const uint32_t key = s.keys[j];
            const float v = __ldg(a.grad + tile0 + key);
            const float av = fabsf(v);
            // L = least k with |v| >= B_k; |v| >= B_tau holds, B is non-increasing in k
            uint32_t lo = 0, hi = a.tau;
            while (lo < hi) {
                const uint32_t mid = (lo + hi) >> 1;
                if (av >= s.thr[mid]) hi = mid; else lo = mid + 1;
            }
            const uint32_t L = lo < 1u ? 1u : lo;
            s.codes[j] = (uint8_t)((v < 0.0f ? 0x80u : 0u) | (L - 1u));
            const uint32_t delta = key - (j ? (uint32_t)s.keys[j - 1] : 0u);
            local_max = max(local_max, delta);
        }
        local_max = __reduce_max_sync(kFullMask, local_max);
        if (lane == 0 && local_max) atomicMax(&s.max_delta, local_max);
    }
    __syncthreads();

    // ---- M, level widths, flags; exclusive scan of the widths; pack
    const uint32_t maxd = s.max_delta;
    const uint32_t M = maxd ? (32u - __clz(maxd)) : 1u;
    const uint32_t levels = 1u << a.l;
    if (tid < (int)levels) s.wtab[tid] = ((tid + 1u) * M + levels - 1u) >> a.l;
    if (tid >= 32 && tid < 32 + 21) {
        const uint32_t bl = tid - 32;                    // flag of a delta of bit length bl
        uint32_t f = 0;
        while (f + 1 < levels && (((f + 1u) * M + levels - 1u) >> a.l) < bl) ++f;
        s.ftab[bl] = f;
    }
    // zero the words the blob can reach
    {
        const uint32_t bound_words = (count * (8u + a.l + M) + 31u) >> 5;
        for (uint32_t i = tid; i < bound_words; i += kEncThreads) s.blob[i] = 0u;
    }
    __syncthreads();

    const uint32_t ipt = (count + kEncThreads - 1) / kEncThreads;   // consecutive keys per thread
    const uint32_t j_lo = min(count, tid * ipt), j_hi = min(count, j_lo + ipt);
    uint32_t my_bits = 0;
    for (uint32_t j = j_lo; j < j_hi; ++j) {
        const uint32_t delta = (uint32_t)s.keys[j] - (j ? (uint32_t)s.keys[j - 1] : 0u);
        my_bits += s.wtab[s.ftab[delta ? 32u - __clz(delta) : 0u]];
    }
    const uint32_t incl = warp_incl_scan(my_bits, lane);
    if (lane == 31) s.scan_tot[warp] = incl;
    __syncthreads();
    uint32_t before = 0, payload_bits = 0;
#pragma unroll
    for (int w = 0; w < kEncWarps; ++w) {
        const uint32_t t = s.scan_tot[w];
        if (w < warp) before += t;
        payload_bits += t;
    }
    const uint32_t flag_pos0 = 8u * count, delta_pos0 = flag_pos0 + a.l * count;
    const uint32_t words = (delta_pos0 + payload_bits + 31u) >> 5;

    // the last warp publishes this group's (count, words) before it packs
    if (warp == kEncWarps - 1 && lane == 0)
        st_release_u64(a.desc + g, desc_pack(g == 0 ? kDescPrefix : kDescAggregate, count, words));

    {
        uint32_t dpos = delta_pos0 + before + (incl - my_bits);
        for (uint32_t j = j_lo; j < j_hi; ++j) {
            const uint32_t delta = (uint32_t)s.keys[j] - (j ? (uint32_t)s.keys[j - 1] : 0u);
            const uint32_t f = s.ftab[delta ? 32u - __clz(delta) : 0u];
            const uint32_t w = s.wtab[f];
            put_bits_smem(s.blob, 8u * j, s.codes[j], 8u);
            put_bits_smem(s.blob, flag_pos0 + a.l * j, f, a.l);
            put_bits_smem(s.blob, dpos, delta, w);
            dpos += w;
        }
    }

    // ---- decoupled look-back (last warp): exclusive prefix of (count, words) over the groups before g
    if (warp == kEncWarps - 1) {
        uint32_t ex_count = 0, ex_words = 0, poisoned = 0;
        if (g > 0) {
            int64_t hi_idx = (int64_t)g - 1;             // window covers hi_idx - lane
            uint32_t spins = 0;
            while (true) {
                const int64_t idx = hi_idx - lane;
                unsigned long long d = idx >= 0 ? ld_acquire_u64(a.desc + idx) : desc_pack(kDescPrefix, 0, 0);
                const uint32_t st = (uint32_t)(d >> 62);
                const uint32_t invalid = __ballot_sync(kFullMask, st == (uint32_t)kDescInvalid);
                const uint32_t poison  = __ballot_sync(kFullMask, st == (uint32_t)kDescPoison);
                const uint32_t prefix  = __ballot_sync(kFullMask, st == (uint32_t)kDescPrefix);
                // lanes are usable up to (not including) the first invalid one
                const uint32_t usable = invalid ? ((1u << (__ffs(invalid) - 1)) - 1u) : kFullMask;
                if (poison & usable) { poisoned = 1; break; }
                const uint32_t pfx_usable = prefix & usable;
                if (pfx_usable) {
                    const int stop = __ffs(pfx_usable) - 1;       // nearest predecessor holding a prefix
                    const bool take = lane <= stop;
                    ex_count += __reduce_add_sync(kFullMask, take ? desc_count(d) : 0u);
                    ex_words += __reduce_add_sync(kFullMask, take ? desc_words(d) : 0u);
                    break;
                }
                if (usable == kFullMask) {                        // 32 aggregates: take them and go on
                    ex_count += __reduce_add_sync(kFullMask, desc_count(d));
                    ex_words += __reduce_add_sync(kFullMask, desc_words(d));
                    hi_idx -= 32;
                    spins = 0;
                    continue;
                }
                // some descriptor in the window is not published yet: take the usable part, wait
                const int nuse = __popc(usable);
                if (nuse) {
                    const bool take = lane < nuse;
                    ex_count += __reduce_add_sync(kFullMask, take ? desc_count(d) : 0u);
                    ex_words += __reduce_add_sync(kFullMask, take ? desc_words(d) : 0u);
                    hi_idx -= nuse;
                    spins = 0;
                    continue;
                }
                if (++spins > kLookbackSpinLimit) { poisoned = 2; break; }
                __nanosleep(64);
            }
        }
        if (lane == 0) {
            if (poisoned) {
                if (poisoned == 2) atomicExch(&a.ctl->error, (unsigned)kStTimeout);
                st_release_u64(a.desc + g, desc_pack(kDescPoison, 0, 0));
            } else if (g > 0) {
                st_release_u64(a.desc + g, desc_pack(kDescPrefix, ex_count + count, ex_words + words));
            }
            s.excl_count = ex_count;
            s.excl_words = ex_words;
            s.poisoned = poisoned;
        }
    }
    __syncthreads();

    // ---- copy-out, directory entry, header
    const uint32_t fixed_words = (kHeaderBytes + 8u * a.G) >> 2;
    const uint32_t off = fixed_words + s.excl_words;
    const uint64_t end_bytes = ((uint64_t)off + words) << 2;
    uint32_t* outw = reinterpret_cast<uint32_t*>(a.out);
    if (!s.poisoned) {
        if (end_bytes <= a.out_bytes)
            for (uint32_t i = tid; i < words; i += kEncThreads) outw[off + i] = bswap32(s.blob[i]);
        if (tid == 0) {
            outw[(kHeaderBytes >> 2) + 2 * g]     = count ? (count | (M << 24)) : 0u;
            outw[(kHeaderBytes >> 2) + 2 * g + 1] = off;
        }
    }
    if (g == a.G - 1 && tid == 0) {
        int status = kStOk;
        const unsigned err = s.poisoned ? (unsigned)kStTimeout : 0u;
        if (err) status = kStTimeout;
        else if (skip == 2u) status = kStNonfinite;
        else if (end_bytes > a.out_bytes) status = kStCapacity;
        const uint64_t d_total = status == kStOk ? (uint64_t)s.excl_count + count : 0ull;
        const uint64_t total = status == kStOk ? end_bytes : (uint64_t)kHeaderBytes;
        const double S = status == kStNonfinite ? 0.0 : a.ctl->sum;
        outw[0] = kMagic;
        outw[1] = kVersion;
        outw[2] = (uint32_t)status;
        outw[3] = a.tau;
        outw[4] = (uint32_t)a.n;            outw[5] = (uint32_t)(a.n >> 32);
        outw[6] = (uint32_t)d_total;        outw[7] = (uint32_t)(d_total >> 32);
        outw[8] = (uint32_t)total;          outw[9] = (uint32_t)(total >> 32);
        const unsigned long long sb = (unsigned long long)__double_as_longlong(S);
        const unsigned long long bb = (unsigned long long)__double_as_longlong(a.base);
        outw[10] = (uint32_t)sb;            outw[11] = (uint32_t)(sb >> 32);
        outw[12] = (uint32_t)bb;            outw[13] = (uint32_t)(bb >> 32);
        outw[14] = a.l | ((uint32_t)kGroupLog2 << 8);
        outw[15] = a.G;
    }
}

}  // namespace fsg
