// The encoder for a gradient given as key-value pairs (Sec. 2.2: the D non-zero pairs (k_j, v_j) of a
// D_m-dimensional gradient): one cooperative launch whose cost follows the number of pairs, not D_m.
//
// The list of pairs is cut into slices of consecutive entries, one per warp.  A warp owns the chunks
// (aligned ranges of 2^14 indices: the unit of the sum tree) and the groups (2^group_log2 indices: one
// instance of Algorithm 2) whose FIRST entry lies in its slice, and follows each to its end, which may lie
// beyond the slice.  Nothing of size D_m is formed: a warp builds, in its own piece of shared memory, the
// 128-entry units of the sum tree that hold entries, and a group's blob straight from the kept entries.
//
//   pass 1  sum (Algorithm 1, first step): per chunk with entries, its node of the fixed fp64 tree.  Zeros add
//           exactly nothing, so only the units with entries are formed: a unit's 128 leaves in shared memory and
//           its node by the usual tree, the 128 unit nodes of the chunk by the same tree one level up.  The
//           chunk nodes go to an array that is zero between launches; the last block to arrive at the grid
//           barrier reduces it on the top of the tree (the very code of the dense encoder), stores S and
//           clears it again.
//   pass 2  sizes: per group with entries, the threshold filter |v| >= B_tau, the delta keys (Eq. 4), their
//           largest (hence M) and a histogram of their bit lengths (hence the payload bits); the group's
//           (count, M, words) is left in the workspace, the block's totals in a table of one entry per block.
//   grid barrier; every block adds up the totals of the blocks before it: its place in the stream.
//   pass 3  pack: per group again, codes || flags || deltas packed in the warp's shared memory (in place in the
//           stream for blobs too long for it), copied out, with the group's directory entry and those of the
//           groups without entries before it.  The owner of the last group with entries writes the header.
//
// Every wait is bounded; when one runs out the block marks the stream FASTSGD_ST_TIMEOUT and leaves.
// Keys that do not ascend or reach n give an unspecified stream, never an access outside the buffers.
#pragma once

#include "common.cuh"
#include "sum.cuh"
#include "bits.cuh"
#include "compress.cuh"     // tree reduction of the partials, table search, flag rule, ordering primitives

namespace fsg {

constexpr int      kKvThreads    = kCmpThreads;      // the shared reduction of the partials is written for this block size
constexpr int      kKvWarps      = kKvThreads / 32;
constexpr uint32_t kKvStageWords = 256;               // blobs up to this many words are packed in shared memory
constexpr uint32_t kKvUnit       = 128;               // leaves of the sum tree formed at a time (4 per lane)
constexpr uint32_t kKvMaxGrid    = 512;               // one thread per block adds up the blocks' totals

struct KvArgs {
    const uint32_t*     keys;        // ascending, each < n
    const float*        vals;        // (DENSE variant: the gradient itself, n floats; keys unused: entry e is (e, vals[e]))
    uint64_t            count;       // D (DENSE variant: n)
    uint64_t            n;           // D_m
    uint8_t*            out;
    uint64_t            out_bytes;
    Control*            ctl;
    double*             partials;    // [chunks], all zero between launches
    unsigned long long* meta;        // [G]: count | M << 24 | words << 32 of the groups with entries
    unsigned long long* blk_agg;     // [gridDim.x]: kept entries << 32 | blob words of each block's groups
    double              base;
    uint32_t            G;           // groups: ceil(n / 2^group_log2)
    uint32_t            chunks;      // ceil(n / 2^14)
    uint32_t            tau;
    uint32_t            l;
    uint32_t            group_log2;
    uint32_t            slice;       // list entries per warp, a multiple of 32
    uint32_t            wait_limit;
    uint32_t            given_sum;   // 1: S is already in the workspace (the list holds kept candidates of a dense gradient); pass 1 is skipped
    // the list was made on the device by k_select_pairs: its length is read from there (kListOverflow: it did not fit)
    const unsigned long long* count_dev;
    uint32_t            run_if;      // 0: always; 1: only if the list fits; 2: only if it does not (the dense walk takes over)
    uint32_t            pad;
};
constexpr unsigned long long kListOverflow = ~0ull;

struct KvWarp {
    float    unit[kKvUnit];          // leaves of the unit being formed; all zero between units
    double   usum[128];              // the chunk's unit nodes (2^14 / 128 of them)
    uint32_t hist[40];               // kept deltas of the group by bit length
    uint32_t stage[kKvStageWords];   // the blob being packed (big-endian valued words)
};

struct KvSmem {
    float    thr[132];
    double   s_tree[kKvWarps];
    double   s_nodes[256];
    unsigned long long scan64[kKvWarps], scan64b[kKvWarps];
    uint32_t wcount[kKvWarps], wwords[kKvWarps];   // pass 2: kept entries and blob words of each warp's groups
    uint32_t flag;                   // block-wide answers of thread 0
    uint32_t abort_flag;
    double   S;
    KvWarp   w[kKvWarps];
};

// Node of the unit at hand -> usum[u]; the leaves return to zero.
__device__ __forceinline__ void kv_flush_unit(KvWarp& ws, uint32_t u, int lane) {
    __syncwarp();
    float4* u4 = reinterpret_cast<float4*>(ws.unit);
    const float4 q = u4[lane];
    u4[lane] = make_float4(0.f, 0.f, 0.f, 0.f);
    const double t = warp_tree(abs_sum4(q));
    if (lane == 0) ws.usum[u] = t;
    __syncwarp();
}

// Pass 1 for the chunk whose first entry is list entry `head`.
__device__ __forceinline__ void kv_sum_chunk(KvWarp& ws, const KvArgs& a, uint64_t head, uint32_t c, int lane) {
#pragma unroll
    for (int i = 0; i < 4; ++i) ws.usum[4 * lane + i] = 0.0;
    __syncwarp();
    uint32_t cur = 0xFFFFFFFFu;
    for (uint64_t base = head;; base += 32u) {
        const uint64_t e = base + (uint64_t)lane;
        uint32_t k = 0u; float v = 0.f;
        if (e < a.count) { k = __ldg(a.keys + e); v = __ldg(a.vals + e); }
        const bool valid = e < a.count && (k >> kChunkLog2) == c;
        const uint32_t vm = __ballot_sync(kFullMask, valid);
        const uint32_t unit = (k >> 7) & 127u;
        uint32_t rem = vm;
        while (rem) {                                     // the units present in this batch, in list order
            const int leader = __ffs((int)rem) - 1;
            const uint32_t u = __shfl_sync(kFullMask, unit, leader);
            const bool mine = valid && unit == u;
            if (u != cur) {
                if (cur != 0xFFFFFFFFu) kv_flush_unit(ws, cur, lane);
                cur = u;
            }
            if (mine) ws.unit[k & 127u] = fabsf(v);
            rem &= ~__ballot_sync(kFullMask, mine);
        }
        if (vm != kFullMask) break;                       // the chunk ended in this batch (or the list did)
    }
    if (cur != 0xFFFFFFFFu) kv_flush_unit(ws, cur, lane);
    const double x = __dadd_rn(__dadd_rn(ws.usum[4 * lane], ws.usum[4 * lane + 1]), __dadd_rn(ws.usum[4 * lane + 2], ws.usum[4 * lane + 3]));
    const double node = warp_tree(x);
    if (lane == 0) a.partials[c] = node;
    __syncwarp();
}

// flag of a delta of bit length bl (0 for a delta of 0): the same rule as flag_of
__device__ __forceinline__ uint32_t kv_flag_of_bl(uint32_t bl, uint32_t l, uint32_t inv_m) {
    return bl ? ((((bl - 1u) << l) * inv_m) >> 16) : 0u;
}

// One batch of 32 list entries of group g starting at list entry `base`: which lanes hold entries of the group, which
// of them are kept, and each kept entry's delta key (Eq. 4; the first of a group counts from g * T).  `prev` is the
// last kept key before the batch and is advanced.
struct KvBatch { uint32_t key; float val; uint32_t vm, km, delta; bool kept; };

// The walk's loads run ahead of their use: the entries of the next kAhead batches are on their way while a batch is
// worked on (a warp walks a group alone, 32 entries per step, and every step would otherwise wait for its own load).
constexpr int kAhead = 4;
template <bool DENSE>
struct KvFeed {
    uint32_t k[kAhead];
    float    v[kAhead];
    uint64_t next;
    __device__ __forceinline__ void load(const KvArgs& a, int slot, uint64_t e) {
        k[slot] = 0u; v[slot] = 0.f;
        if (e < a.count) { k[slot] = DENSE ? (uint32_t)e : __ldg(a.keys + e); v[slot] = __ldg(a.vals + e); }
    }
    __device__ __forceinline__ void start(const KvArgs& a, uint64_t base, int lane) {
#pragma unroll
        for (int i = 0; i < kAhead; ++i) load(a, i, base + 32u * (uint32_t)i + (uint64_t)lane);
        next = base + 32u * (uint32_t)kAhead;
    }
    __device__ __forceinline__ void pop(const KvArgs& a, int lane, uint32_t& key, float& val) {
        key = k[0]; val = v[0];
#pragma unroll
        for (int i = 0; i + 1 < kAhead; ++i) { k[i] = k[i + 1]; v[i] = v[i + 1]; }
        load(a, kAhead - 1, next + (uint64_t)lane);
        next += 32u;
    }
};

template <bool DENSE>
__device__ __forceinline__ KvBatch kv_batch(const KvArgs& a, KvFeed<DENSE>& feed, uint64_t base, uint32_t g, float thr_e, uint32_t& prev, int lane) {
    KvBatch b;
    const uint64_t e = base + (uint64_t)lane;
    feed.pop(a, lane, b.key, b.val);
    const bool valid = e < a.count && (b.key >> a.group_log2) == g;
    b.vm = __ballot_sync(kFullMask, valid);
    b.kept = valid && fabsf(b.val) >= thr_e;              // (thr_e is at least the smallest denormal: zeros are never kept; +inf when nothing may be kept)
    b.km = __ballot_sync(kFullMask, b.kept);
    const uint32_t lower = b.km & ((1u << lane) - 1u);
    const int src = lower ? 31 - __clz((int)lower) : 0;
    const uint32_t pk = __shfl_sync(kFullMask, b.key, src);
    b.delta = b.kept ? b.key - (lower ? pk : prev) : 0u;
    if (b.km) prev = __shfl_sync(kFullMask, b.key, 31 - __clz((int)b.km));
    return b;
}

// Pass 2 for the group whose first entry is list entry `head`: count | M << 24 | words << 32.
template <bool DENSE>
__device__ __forceinline__ unsigned long long kv_group_sizes(KvWarp& ws, const KvArgs& a, float thr_e, uint64_t head, uint32_t g, int lane) {
    ws.hist[lane] = 0u;
    if (lane < 8) ws.hist[32 + lane] = 0u;
    __syncwarp();
    uint32_t prev = g << a.group_log2, count = 0u, maxd = 0u;
    KvFeed<DENSE> feed;
    feed.start(a, head, lane);
    for (uint64_t base = head;; base += 32u) {
        const KvBatch b = kv_batch<DENSE>(a, feed, base, g, thr_e, prev, lane);
        if (b.kept) {
            atomicAdd(&ws.hist[b.delta ? 32 - __clz((int)b.delta) : 0], 1u);
            maxd = max(maxd, b.delta);
        }
        count += (uint32_t)__popc(b.km);
        if (b.vm != kFullMask) break;
    }
    maxd = __reduce_max_sync(kFullMask, maxd);
    uint32_t M = maxd ? 32u - (uint32_t)__clz((int)maxd) : 1u;
    M = min(M, 20u);                                      // (more only with keys that do not ascend)
    __syncwarp();
    // payload bits exactly as pass 3 lays them out: a delta of bit length bl takes the width of its (clamped) level;
    // bit length 32 (only with keys that do not ascend) takes the top level, like every length above M
    const uint32_t f = kv_flag_of_bl((uint32_t)lane, a.l, c_inv_m[M]);
    const uint32_t w = ((min(f, (1u << a.l) - 1u) + 1u) * M + (1u << a.l) - 1u) >> a.l;
    const uint32_t bits = __reduce_add_sync(kFullMask, ws.hist[lane] * w + (lane == 0 ? ws.hist[32] * M : 0u));
    __syncwarp();
    if (count > (1u << 20)) count = 0u;                   // more entries than a group has indices (keys that repeat): an empty group
    const uint32_t words = count ? (count * (8u + a.l) + bits + 31u) >> 5 : 0u;
    return (unsigned long long)(count ? (count | (M << 24)) : 0u) | ((unsigned long long)words << 32);
}

// Pass 3 for the same group: its blob written to dst[0, words) (little-endian words of the stream).
template <bool DENSE>
__device__ __forceinline__ void kv_group_pack(KvWarp& ws, const KvArgs& a, const float* thr, uint64_t head, uint32_t g,
                                              uint32_t count, uint32_t M, uint32_t words, uint32_t* dst, int lane) {
    const bool in_smem = words <= kKvStageWords;
    uint32_t* blob = in_smem ? ws.stage : dst;
    for (uint32_t i = lane; i < words; i += 32u) blob[i] = 0u;
    if (!in_smem) __threadfence();
    __syncwarp();
    const float thr_e = thr[a.tau];
    const uint32_t inv_m = c_inv_m[M], round_up = (1u << a.l) - 1u;
    const uint32_t flag_pos0 = 8u * count;
    uint32_t prev = g << a.group_log2, rank = 0u, dpos = flag_pos0 + a.l * count;
    KvFeed<DENSE> feed;
    feed.start(a, head, lane);
    for (uint64_t base = head;; base += 32u) {
        const KvBatch b = kv_batch<DENSE>(a, feed, base, g, thr_e, prev, lane);
        uint32_t f = 0u, w = 0u;
        if (b.kept) {
            f = min(flag_of(b.delta, a.l, inv_m), round_up);
            w = ((f + 1u) * M + round_up) >> a.l;
        }
        const uint32_t w_incl = warp_incl_scan(w, lane);
        // (count, M and words come from the workspace entry of the group; with keys that do not ascend a group can have
        // several first entries and the entry may be another one's: no field is written outside [0, 32 words))
        const uint32_t q = rank + (uint32_t)__popc(b.km & ((1u << lane) - 1u));
        if (b.kept && q < count && dpos + w_incl <= 32u * words) {
            const uint32_t code = code_byte_of(thr, a.tau, b.val);
            const uint32_t d = w >= 32u ? b.delta : (b.delta & ((1u << w) - 1u));
            if (in_smem) {
                put_byte_smem(blob, q, code);
                put_bits_smem(blob, flag_pos0 + a.l * q, f, a.l);
                put_bits_smem(blob, dpos + (w_incl - w), d, w);
            } else {
                // in place: the words of the stream are the byte-swapped big-endian valued words
                atomicOr(&blob[q >> 2], bswap32(code << (24u - 8u * (q & 3u))));
                {
                    const uint32_t pos = flag_pos0 + a.l * q, wi = pos >> 5, sh = pos & 31u;
                    const unsigned long long win = (unsigned long long)f << (64u - sh - a.l);
                    atomicOr(&blob[wi], bswap32((uint32_t)(win >> 32)));
                    if ((uint32_t)win) atomicOr(&blob[wi + 1], bswap32((uint32_t)win));
                }
                if (w) {
                    const uint32_t pos = dpos + (w_incl - w), wi = pos >> 5, sh = pos & 31u;
                    const unsigned long long win = (unsigned long long)d << (64u - sh - w);
                    atomicOr(&blob[wi], bswap32((uint32_t)(win >> 32)));
                    if ((uint32_t)win) atomicOr(&blob[wi + 1], bswap32((uint32_t)win));
                }
            }
        }
        rank += (uint32_t)__popc(b.km);
        dpos = min(dpos + __shfl_sync(kFullMask, w_incl, 31), 32u * words + 1u);      // (beyond the blob only on inconsistent input: stays there)
        if (b.vm != kFullMask) break;
    }
    __syncwarp();
    if (in_smem)
        for (uint32_t i = lane; i < words; i += 32u) dst[i] = bswap32(blob[i]);
}

// Header of the stream; one thread.
__device__ __forceinline__ void kv_write_header(const KvArgs& a, int status, uint64_t d_total, uint64_t total_bytes, double S) {
    uint32_t* outw = reinterpret_cast<uint32_t*>(a.out);
    const uint64_t d = status == kStOk ? d_total : 0ull;
    const uint64_t total = status == kStOk ? total_bytes : (uint64_t)kHeaderBytes;
    const double Sh = (status == kStNonfinite || status == kStTimeout) ? 0.0 : S;
    outw[0] = kMagic; outw[1] = kVersion; outw[2] = (uint32_t)status; outw[3] = a.tau;
    outw[4] = (uint32_t)a.n; outw[5] = (uint32_t)(a.n >> 32);
    outw[6] = (uint32_t)d; outw[7] = (uint32_t)(d >> 32);
    outw[8] = (uint32_t)total; outw[9] = (uint32_t)(total >> 32);
    const unsigned long long sb = (unsigned long long)__double_as_longlong(Sh), bb = (unsigned long long)__double_as_longlong(a.base);
    outw[10] = (uint32_t)sb; outw[11] = (uint32_t)(sb >> 32);
    outw[12] = (uint32_t)bb; outw[13] = (uint32_t)(bb >> 32);
    outw[14] = a.l | (a.group_log2 << 8);
    outw[15] = a.G;
}

// Grid barrier `which` (0 or 1) of the launch, first half.  Returns true in every thread of the one block that
// arrived last (it sets the flag itself once it has done what everybody waits for).
__device__ __forceinline__ bool kv_barrier_arrive(KvSmem& s, Control* ctl, int which, int tid) {
    __syncthreads();
    if (tid == 0) {
        s.flag = 0u;
        if (!s.abort_flag) s.flag = atom_add_acq_rel_u32(&ctl->bar_count[which], 1u) == gridDim.x - 1u ? 1u : 0u;
    }
    __syncthreads();
    return s.flag != 0u;
}
__device__ __forceinline__ void kv_barrier_release(Control* ctl, int which, unsigned int gen_next) {
    ctl->bar_count[which] = 0u;
    st_release_u32(&ctl->bar_flag[which], gen_next);
}
__device__ __forceinline__ void kv_barrier_wait(KvSmem& s, Control* ctl, int which, unsigned int gen_next, uint32_t limit, int tid) {
    if (tid == 0 && !s.abort_flag) {
        uint32_t spin = 0;
        while (ld_acquire_u32(&ctl->bar_flag[which]) != gen_next) {
            if (++spin > limit) { s.abort_flag = 1u; break; }
            if (spin > 64u) __nanosleep(32);
        }
    }
    __syncthreads();
}

// Calls f(head entry, group or chunk number, key of the entry before the head or 0xFFFFFFFF) for every unit of 2^shift
// indices whose first entry lies in the warp's slice [lo, hi) of the list, in list order.  DENSE: the slice counts units,
// unit u starts at entry u << shift and has no gap before it.
template <bool DENSE, typename F>
__device__ __forceinline__ void kv_for_each_head(const KvArgs& a, uint64_t lo, uint64_t hi, uint32_t shift, uint32_t limit, int lane, F f) {
    if (DENSE) {
        for (uint64_t u = lo; u < hi; ++u) f(u << shift, (uint32_t)u, u ? (uint32_t)((u << shift) - 1u) : 0xFFFFFFFFu);
        return;
    }
    for (uint64_t base = lo; base < hi; base += 32u) {
        const uint64_t e = base + (uint64_t)lane;
        uint32_t k = 0u, kp = 0xFFFFFFFFu;
        if (e < hi) { k = __ldg(a.keys + e); if (e) kp = __ldg(a.keys + e - 1); }
        const bool head = e < hi && (e == 0 || (kp >> shift) != (k >> shift)) && (k >> shift) < limit;
        uint32_t hm = __ballot_sync(kFullMask, head);
        while (hm) {
            const int src = __ffs((int)hm) - 1;
            hm &= hm - 1u;
            f(base + (uint64_t)src, __shfl_sync(kFullMask, k, src) >> shift, __shfl_sync(kFullMask, kp, src));
        }
    }
}

// DENSE = false: fastsgd_compress_kv.  DENSE = true: the same passes 2 and 3 over a dense gradient whose sum is already
// in the workspace (group sizes other than the fused encoder's): every index is a list entry, a warp owns a run of groups.
template <bool DENSE>
__global__ void __launch_bounds__(kKvThreads, 2)
k_compress_kv(const KvArgs a_in, const __grid_constant__ PowTable pw) {
    KvArgs a = a_in;
    if (a.count_dev != nullptr) {
        const unsigned long long cnt = __ldcg(a.count_dev);
        if ((a.run_if == 1u && cnt == kListOverflow) || (a.run_if == 2u && cnt != kListOverflow)) return;      // (the same answer in every block)
        if (!DENSE) {
            a.count = cnt;
            const uint64_t warps = (uint64_t)gridDim.x * kKvWarps;
            a.slice = (uint32_t)max((((cnt + warps - 1) / warps) + 31ull) & ~31ull, 32ull);
        }
    }
    extern __shared__ __align__(128) unsigned char kv_smem_raw[];
    KvSmem& s = *reinterpret_cast<KvSmem*>(kv_smem_raw);
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    KvWarp& ws = s.w[warp];
    uint32_t* outw = reinterpret_cast<uint32_t*>(a.out);
    const uint32_t fixed_words = (kHeaderBytes + 8u * a.G) >> 2;

    unsigned int gen_next = 0u;
    if (tid == 0) {
        gen_next = ld_acquire_u32(&a.ctl->bar_gen) + 1u;      // before this block can arrive at a barrier
        s.abort_flag = 0u;
        s.flag = gen_next;
    }
    for (uint32_t i = lane; i < kKvUnit; i += 32u) ws.unit[i] = 0.f;
    __syncthreads();
    gen_next = s.flag;

    // this warp's slice of the list (DENSE: of the groups)
    const uint64_t gw = (uint64_t)blockIdx.x * kKvWarps + (uint64_t)warp;
    const uint64_t units = DENSE ? (uint64_t)a.G : a.count;
    const uint64_t lo = min(units, gw * (uint64_t)a.slice), hi = min(units, lo + (uint64_t)a.slice);

    // ---- pass 1: the chunks whose first entry lies in the slice
    if (!DENSE && !a.given_sum) {
        kv_for_each_head<false>(a, lo, hi, (uint32_t)kChunkLog2, a.chunks, lane,
                                [&](uint64_t head_e, uint32_t c, uint32_t) { kv_sum_chunk(ws, a, head_e, c, lane); });
        // ---- grid barrier; the last block to arrive reduces the chunk nodes (same tree, same code as the dense encoder)
        if (kv_barrier_arrive(s, a.ctl, 0, tid)) {
            const double S = a.chunks > kCmpBigTiles ? reduce_partials<true>(a.partials, a.chunks, s.s_tree, s.s_nodes, tid, lane, warp)
                                                     : reduce_partials<false>(a.partials, a.chunks, s.s_tree, s.s_nodes, tid, lane, warp);
            __syncthreads();
            for (uint32_t i = tid; i < a.chunks; i += kKvThreads) a.partials[i] = 0.0;     // at rest again
            __syncthreads();
            if (tid == 0) {
                __threadfence();
                reinterpret_cast<double*>(reinterpret_cast<unsigned char*>(a.ctl) + kJobSumOffset)[0] = S;
                kv_barrier_release(a.ctl, 0, gen_next);
            }
        }
        kv_barrier_wait(s, a.ctl, 0, gen_next, a.wait_limit, tid);
    }

    // ---- boundary table RU32(B_k), as the dense encoder forms it
    if (tid == 0) s.S = __ldcg(reinterpret_cast<const double*>(reinterpret_cast<const unsigned char*>(a.ctl) + kJobSumOffset));
    __syncthreads();
    const double S = s.S;
    const bool finite = isfinite(S);
    if (tid <= (int)a.tau)
        s.thr[tid] = (finite && S != 0.0) ? fmaxf(__double2float_ru(__ddiv_rn(S, pw.P[tid])), __int_as_float(1)) : __int_as_float(0x7f800000);
    if (tid == 0) {                                       // (estimates that only steer the table search: see make_table)
        const unsigned long long sb = (unsigned long long)__double_as_longlong(S);
        const float mant = __uint_as_float(0x3F800000u | (uint32_t)((sb >> 29) & 0x7FFFFFull));
        s.thr[130] = (float)((int)((sb >> 52) & 0x7FFull) - 1023) + __log2f(mant);
        s.thr[131] = 1.0f / __log2f((float)a.base);
    }
    __syncthreads();
    const float thr_e = s.thr[a.tau];
    const bool aborted1 = s.abort_flag != 0u;

    // ---- pass 2: sizes of the groups whose first entry lies in the slice
    uint32_t my_count = 0u, my_words = 0u;
    if (!aborted1) {
        kv_for_each_head<DENSE>(a, lo, hi, a.group_log2, a.G, lane, [&](uint64_t head_e, uint32_t g, uint32_t) {
            const unsigned long long m = kv_group_sizes<DENSE>(ws, a, thr_e, head_e, g, lane);
            if (lane == 0) a.meta[g] = m;
            my_count += (uint32_t)m & 0xFFFFFFu;
            my_words += (uint32_t)(m >> 32);
        });
    }
    if (lane == 0) { s.wcount[warp] = my_count; s.wwords[warp] = my_words; }
    __syncthreads();
    if (tid == 0) {
        unsigned long long agg = 0ull;
        for (int w = 0; w < kKvWarps; ++w) agg += ((unsigned long long)s.wcount[w] << 32) | s.wwords[w];
        st_relaxed_u64(a.blk_agg + blockIdx.x, agg);
    }
    // ---- grid barrier; then every block adds up the totals of the blocks before it
    if (kv_barrier_arrive(s, a.ctl, 1, tid)) {
        if (tid == 0) kv_barrier_release(a.ctl, 1, gen_next);
    }
    kv_barrier_wait(s, a.ctl, 1, gen_next, a.wait_limit, tid);
    const bool aborted = s.abort_flag != 0u;

    if (!aborted) {
        unsigned long long mine = (uint32_t)tid < gridDim.x ? ld_relaxed_u64(a.blk_agg + tid) : 0ull;
        unsigned long long before = (uint32_t)tid < blockIdx.x ? mine : 0ull;
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) {
            mine += __shfl_xor_sync(kFullMask, mine, o);
            before += __shfl_xor_sync(kFullMask, before, o);
        }
        __syncthreads();
        if (lane == 0) { s.scan64[warp] = mine; s.scan64b[warp] = before; }
        __syncthreads();
        unsigned long long all = 0ull, base_blk = 0ull;
#pragma unroll
        for (int w = 0; w < kKvWarps; ++w) { all += s.scan64[w]; base_blk += s.scan64b[w]; }
        for (int w = 0; w < warp; ++w) base_blk += ((unsigned long long)s.wcount[w] << 32) | s.wwords[w];
        const uint64_t d_total = all >> 32;
        const uint32_t words_total = (uint32_t)all;
        const uint64_t total_bytes = ((uint64_t)fixed_words + words_total) << 2;
        int status = kStOk;
        if (!finite) status = kStNonfinite;
        else if (total_bytes > a.out_bytes) status = kStCapacity;
        const bool write_blobs = status == kStOk;

        // ---- pass 3: the same groups again: directory entries, blobs, header
        uint32_t off = fixed_words + (uint32_t)base_blk;          // word offset of the next blob of this warp
        kv_for_each_head<DENSE>(a, lo, hi, a.group_log2, a.G, lane, [&](uint64_t head_e, uint32_t g, uint32_t kprev) {
            const unsigned long long m = __ldcg(a.meta + g);
            const uint32_t cm = (uint32_t)m, count = cm & 0xFFFFFFu, M = cm >> 24, words = (uint32_t)(m >> 32);
            // the groups without entries between the last group with entries and this one start where this one does
            const uint32_t gap0 = head_e ? min((kprev >> a.group_log2) + 1u, g) : 0u;
            for (uint32_t gg = gap0 + (uint32_t)lane; gg < g; gg += 32u) {
                outw[(kHeaderBytes >> 2) + 2u * gg] = 0u;
                outw[(kHeaderBytes >> 2) + 2u * gg + 1u] = off;
            }
            if (lane == 0) {
                outw[(kHeaderBytes >> 2) + 2u * g] = cm;
                outw[(kHeaderBytes >> 2) + 2u * g + 1u] = off;
            }
            if (count && write_blobs && M >= 1u && M <= 20u && (uint64_t)count * (8u + a.l) <= 32ull * words &&
                (uint64_t)off + words <= (uint64_t)fixed_words + words_total)
                kv_group_pack<DENSE>(ws, a, s.thr, head_e, g, count, M, words, outw + off, lane);
            off = (uint32_t)min((uint64_t)off + words, (uint64_t)fixed_words + words_total);
        });
        // block 0: the groups after the last one with entries (they start where the stream ends), and the header
        if (blockIdx.x == 0) {
            uint32_t g_end = 0u;
            if (DENSE) g_end = a.G;
            else if (a.count) g_end = min(a.G, (__ldg(a.keys + a.count - 1) >> a.group_log2) + 1u);
            for (uint32_t gg = g_end + (uint32_t)tid; gg < a.G; gg += kKvThreads) {
                outw[(kHeaderBytes >> 2) + 2u * gg] = 0u;
                outw[(kHeaderBytes >> 2) + 2u * gg + 1u] = fixed_words + words_total;
            }
            if (tid == 0) kv_write_header(a, status, d_total, total_bytes, S);
        }
    }

    if (s.abort_flag) {
        __syncthreads();
        if (tid == 0) {
            atomicExch(&a.ctl->error, (unsigned)kStTimeout);
            kv_write_header(a, kStTimeout, 0ull, 0ull, 0.0);
        }
    }
    // the last block to leave readies the workspace for the next launch (and has the final word on a timeout)
    __syncthreads();
    if (tid == 0) {
        const unsigned int old = atom_add_acq_rel_u32(&a.ctl->exit_count, 1u);
        if (old == gridDim.x - 1u) {
            if (ld_acquire_u32(&a.ctl->error) != 0u) kv_write_header(a, kStTimeout, 0ull, 0ull, 0.0);
            a.ctl->exit_count = 0u;
            st_release_u32(&a.ctl->bar_gen, gen_next);
        }
    }
}


// Dense gradient -> the list of its kept entries (i, v_i), |v_i| >= B_tau, in index order, for the list encoder:
// the general path of fastsgd_compress for group sizes other than the fused kernel's.  One cooperative launch: every
// warp counts the kept entries of its contiguous share of the gradient, the blocks' totals meet at a grid barrier,
// every warp then writes its entries behind those of the warps before it.  S is in the workspace (k_abs_sum).  If
// the list does not fit `capacity` pairs, *count_out = kListOverflow and nothing is written.
struct SelArgs {
    const float*        grad;
    uint64_t            n;
    Control*            ctl;
    unsigned long long* blk_agg;     // [gridDim.x]
    uint32_t*           keys;        // [capacity]
    float*              vals;        // [capacity]
    unsigned long long* count_out;
    uint64_t            capacity;
    uint32_t            tau;
    uint32_t            wait_limit;
};

__global__ void __launch_bounds__(kKvThreads, 2)
k_select_pairs(const SelArgs a, const __grid_constant__ PowTable pw) {
    __shared__ uint32_t s_w[kKvWarps];
    __shared__ unsigned long long s_scan[kKvWarps], s_scanb[kKvWarps];
    __shared__ uint32_t s_flag, s_abort;
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    unsigned int gen_next = 0u;
    if (tid == 0) { s_flag = ld_acquire_u32(&a.ctl->bar_gen) + 1u; s_abort = 0u; }
    __syncthreads();
    gen_next = s_flag;
    const double S = __ldcg(reinterpret_cast<const double*>(reinterpret_cast<const unsigned char*>(a.ctl) + kJobSumOffset));
    const float thr_e = (isfinite(S) && S != 0.0) ? fmaxf(__double2float_ru(__ddiv_rn(S, pw.P[a.tau])), __int_as_float(1)) : __int_as_float(0x7f800000);
    // this warp's share: whole steps of 128 entries (a float4 per lane)
    const uint64_t steps = (a.n + 127ull) >> 7;
    const uint64_t warps = (uint64_t)gridDim.x * kKvWarps, gw = (uint64_t)blockIdx.x * kKvWarps + (uint64_t)warp;
    const uint64_t per = (steps + warps - 1) / warps;
    const uint64_t s0 = min(steps, gw * per), s1 = min(steps, s0 + per);
    auto mask_of = [&](uint64_t step) -> uint32_t {
        const float4 q = load4_guarded(a.grad, (step << 7) + 4ull * (uint64_t)lane, a.n);
        return (fabsf(q.x) >= thr_e ? 1u : 0u) | (fabsf(q.y) >= thr_e ? 2u : 0u) | (fabsf(q.z) >= thr_e ? 4u : 0u) | (fabsf(q.w) >= thr_e ? 8u : 0u);
    };
    uint32_t mine = 0u;
    for (uint64_t st = s0; st < s1; ++st) mine += (uint32_t)__popc(mask_of(st));
    mine = __reduce_add_sync(kFullMask, mine);
    if (lane == 0) s_w[warp] = mine;
    __syncthreads();
    if (tid == 0) {
        unsigned long long tot = 0ull;
        for (int w = 0; w < kKvWarps; ++w) tot += s_w[w];
        st_relaxed_u64(a.blk_agg + blockIdx.x, tot);
        // grid barrier (the launch's only one): the last block to arrive opens it
        if (atom_add_acq_rel_u32(&a.ctl->bar_count[0], 1u) == gridDim.x - 1u) {
            a.ctl->bar_count[0] = 0u;
            st_release_u32(&a.ctl->bar_flag[0], gen_next);
        }
        uint32_t spin = 0;
        while (ld_acquire_u32(&a.ctl->bar_flag[0]) != gen_next) {
            if (++spin > a.wait_limit) { s_abort = 1u; break; }
            if (spin > 64u) __nanosleep(32);
        }
    }
    __syncthreads();
    if (!s_abort) {
        unsigned long long all = (uint32_t)tid < gridDim.x ? ld_relaxed_u64(a.blk_agg + tid) : 0ull;
        unsigned long long before = (uint32_t)tid < blockIdx.x ? all : 0ull;
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) {
            all += __shfl_xor_sync(kFullMask, all, o);
            before += __shfl_xor_sync(kFullMask, before, o);
        }
        if (lane == 0) { s_scan[warp] = all; s_scanb[warp] = before; }
        __syncthreads();
        unsigned long long total = 0ull, base = 0ull;
#pragma unroll
        for (int w = 0; w < kKvWarps; ++w) { total += s_scan[w]; base += s_scanb[w]; }
        for (int w = 0; w < warp; ++w) base += s_w[w];
        const bool fits = total <= a.capacity;
        if (blockIdx.x == 0 && tid == 0) *a.count_out = fits ? total : kListOverflow;
        if (fits) {
            unsigned long long pos = base;
            for (uint64_t st = s0; st < s1; ++st) {
                const uint64_t e0 = (st << 7) + 4ull * (uint64_t)lane;
                const float4 q = load4_guarded(a.grad, e0, a.n);
                const uint32_t m = (fabsf(q.x) >= thr_e ? 1u : 0u) | (fabsf(q.y) >= thr_e ? 2u : 0u) | (fabsf(q.z) >= thr_e ? 4u : 0u) | (fabsf(q.w) >= thr_e ? 8u : 0u);
                const uint32_t c = (uint32_t)__popc(m);
                const uint32_t incl = warp_incl_scan(c, lane);
                unsigned long long p = pos + (incl - c);
                if (m & 1u) { a.keys[p] = (uint32_t)e0;      a.vals[p] = q.x; ++p; }
                if (m & 2u) { a.keys[p] = (uint32_t)e0 + 1u; a.vals[p] = q.y; ++p; }
                if (m & 4u) { a.keys[p] = (uint32_t)e0 + 2u; a.vals[p] = q.z; ++p; }
                if (m & 8u) { a.keys[p] = (uint32_t)e0 + 3u; a.vals[p] = q.w; ++p; }
                pos += __shfl_sync(kFullMask, incl, 31);
            }
        }
    } else if (blockIdx.x == 0 && tid == 0) {
        *a.count_out = kListOverflow;                     // (a wait ran out: the dense walk takes over; the next launch's waits report it)
    }
    // the last block to leave bumps the generation
    __syncthreads();
    if (tid == 0) {
        const unsigned int old = atom_add_acq_rel_u32(&a.ctl->exit_count, 1u);
        if (old == gridDim.x - 1u) {
            a.ctl->exit_count = 0u;
            st_release_u32(&a.ctl->bar_gen, gen_next);
        }
    }
}

}  // namespace fsg
