// The encoder as ONE persistent kernel (two thread blocks per SM, cooperative launch) that takes up
// to eight gradients of the same length.
//
// Sum pass (Algorithm 1, first step): tiles of 2^14 entries, handed out by a ticket counter, go
// through a 64 KiB shared-memory stage in four parts filled by bulk asynchronous copies (TMA, no
// multicast): one part is summed while the other three are in flight.  Each tile is reduced on the fixed
// fp64 pairwise tree; one partial and the tile's largest |v| are left in the workspace.  Grid
// barrier (bounded wait).  The last block to arrive reduces all partials in the same tree order,
// stores the sum and lists the tiles whose largest |v| reaches the early-stop threshold.
// Encode pass (rest of Algorithm 1, Algorithm 2 per group): blocks take the listed tiles by ticket
// (the others hold nothing to keep and are not read again); the next tile's copy runs while the
// block filters, compacts, quantises, delta-encodes and bit-packs the tile at hand, every warp on
// its own slab of 1024 entries, with two block barriers per tile.
//
// Device-wide offsets.  A packed blob stays in a shared-memory arena and the tile's
// (count, words) is published as a descriptor; no block waits for another while it packs.
// When the arena fills up the block drains it: it brings its running exclusive scan of all
// descriptors up to its pending tiles (block-wide shuffle scans over 4 x 512 descriptors at a
// time, bounded polls for the ones not published yet), copies the blobs to their places in the
// stream and writes their directory entries.  A block never waits while it holds a reserved tile,
// and the block that owns the lowest unpublished tile never waits for anything, so the scheme
// cannot deadlock provided all blocks are resident (cooperative launch).  What is pending at the
// end of a gradient's encode pass is placed from prefixes that one block computes for everybody.
// Every wait is bounded; when one runs out the block records FASTSGD_ST_TIMEOUT, poisons its
// descriptors, waits (bounded) for its own copies in flight and returns.
#pragma once

#include "common.cuh"
#include "sum.cuh"
#include "bits.cuh"

namespace fsg {

constexpr int      kCmpThreads   = 512;
constexpr int      kCmpWarps     = kCmpThreads / 32;
constexpr int      kStages       = 1;
constexpr int      kSumParts     = 2;                         // the sum pass brings a tile in as this many parts, each with its own copy and barrier (4: measured 8 % slower on 4 x 25.6 M entries, 3 % on 2^28: more barriers and shuffles per tile than the extra copies in flight pay for)
constexpr uint32_t kPartEntries  = (1u << kGroupLog2) / kSumParts;
constexpr int      kPartRows     = (int)(kPartEntries / (uint32_t)kCmpWarps / 128u);   // rows of 128 entries a warp sums per part
static_assert(kPartRows == 2 || kPartRows == 4, "a warp sums two or four rows of 128 entries per part");
constexpr uint32_t kTile         = 1u << kGroupLog2;          // entries per tile = per group
constexpr uint32_t kSlabCap      = 192;                       // kept entries a warp's 1024-entry slab may have on the shared-memory path
constexpr uint32_t kArenaWords   = 4608;                      // packed blobs waiting for their offsets
constexpr int      kPendMax      = 128;                       // tiles that may wait in the arena
constexpr uint32_t kArenaReserve = 1024;                      // drain ahead of time when less than this would be left
constexpr uint32_t kMaxCtas      = 320;                       // scratch slots for the dense path
constexpr uint32_t kWaitLimit    = 1u << 22;                  // polls before a wait gives up
constexpr int      kDrainChunks  = 4;                         // descriptors read at once when draining: 4 x 512
constexpr uint32_t kNoTicket     = 0xFFFFFFFEu;               // "no tile reserved": the block drains before it takes one
constexpr uint32_t kNoMore       = 0xFFFFFFFDu;               // "no tile left": the gradient's list is exhausted
constexpr uint32_t kDenseMark    = 0xFFFFFFFFu;               // arena offset of a blob that sits in global scratch
// dense path scratch per block: values / blob u32[T] | keys u16[T] | codes u8[T]
constexpr uint64_t kDenseScratchBytes = (uint64_t)kTile * 4u + (uint64_t)kTile * 2u + kTile;
static_assert(kArenaWords >= (kCmpWarps * kSlabCap * (8u + 5u + 14u) + 31u) / 32u, "arena holds the widest sparse blob");

constexpr unsigned long long kDescValid = 1ull;               // status of a published descriptor (kDescPoison = 3)

struct CmpSmem {
    float    stage[kStages][kTile];
    unsigned long long mbar[kSumParts];      // [0]: the whole tile (encode pass); [p]: part p of the tile (sum pass)
    double   s_warp[2][kSumParts][kCmpWarps];// sum pass, by tile parity and part: the warps' tree nodes
    uint32_t s_wmax[2][kSumParts][kCmpWarps];// ... and largest |v| (bits of a non-negative float)
    double   s_tree[kCmpWarps];
    unsigned long long scan64[kDrainChunks][kCmpWarps];
    float    thr[132];
    // per-slab summaries, by tile parity (an empty tile has no second barrier)
    uint32_t sum_count[2][kCmpWarps];        // kept entries of the slab; bit 31: more than kSlabCap
    uint32_t sum_first[2][kCmpWarps];        // first and last kept key (tile-local) of the slab
    uint32_t sum_last[2][kCmpWarps];
    uint32_t sum_maxd[2][kCmpWarps];         // largest delta between two kept keys of the slab
    uint32_t sum_bits[2][kCmpWarps];         // payload bits of the slab
    uint32_t scan_tot[kCmpWarps];
    uint32_t scan_tot2[2][kCmpWarps];
    uint32_t pend_g[kPendMax];
    uint32_t pend_cm[kPendMax];              // count | M << 24
    uint32_t pend_words[kPendMax];
    uint32_t pend_off[kPendMax];             // word offset in the arena, or kDenseMark
    unsigned long long pend_prefix[kPendMax];// exclusive prefix: count << 32 | words
    uint32_t max_delta;
    uint32_t abort_flag;
    uint32_t poison_seen;
    uint32_t wait_limit;                     // polls before a wait on another block gives up (from the launch arguments)
    uint32_t next_tile[2];                   // by tile parity: the tile this block works on next
    uint32_t ne_count;                       // tiles the gradient's encode pass hands out by ticket
    uint32_t try_limit;                      // tries before a wait on a bulk copy gives up (from the launch arguments)
    uint32_t held[2];                        // tiles this block has taken and not yet published (for the give-up path)
    uint32_t sc_pos, sc_count, sc_words;     // running exclusive scan of the descriptors: [0, pos) included
    uint32_t job_skip[2];                    // by gradient parity: 0 encode, 1 sum == 0, 2 sum not finite
    double   job_sum[2];                     // by gradient parity: its sum
    double   s_nodes[256];                   // nodes of the final sum tree when a thread holds more than 8 partials
    uint32_t pad5;                           // (scratch flag of the shared descriptor scan)
    uint32_t publisher;                      // this block was the last to finish the gradient's encode pass
    uint32_t team;                           // which of the two teams of blocks this one belongs to
    uint32_t last_arrival;                   // this block was the last to arrive at a grid barrier
    uint32_t p1_next[2];                     // the same for the sum pass
    uint32_t arena[kArenaWords];
    uint32_t wvals[kCmpWarps][kSlabCap];     // per warp: kept values (fp32 bits), then their code bytes
    uint16_t wkeys[kCmpWarps][kSlabCap];     // per warp: kept keys (tile-local), in index order
};
static_assert(sizeof(CmpSmem) <= 232448, "shared memory of one block on sm_100");
static_assert(2 * (sizeof(CmpSmem) + 1024) <= 233472, "two blocks per SM (1 KiB per block is the system's)");

constexpr int kCmpMaxJobs = 8;             // gradients (simulated workers) one launch can take
constexpr uint32_t kCmpBigTiles = 8192;   // a single gradient with more tiles than this is compressed by the kernel variant for very many tiles

// One gradient's view of the launch arguments.
struct CmpArgs {
    const float*        grad;
    uint64_t            n;
    uint8_t*            out;
    uint64_t            out_bytes;
    Control*            ctl;
    unsigned int*       ticket;          // this gradient's tile counter of the encode pass
    double*             partials;
    unsigned long long* desc;
    unsigned long long* prefix;          // exclusive scan of desc, written by the last block to finish the encode pass
    float*              tmax;            // largest |v| of each tile, from the sum pass
    uint32_t*           nelist;          // the tiles the encode pass reads, ascending: those whose largest |v| reaches the threshold
    uint32_t*           nebits;          // the same as a bitmap (scratch of the block that builds the list)
    unsigned int*       enc_done;        // blocks that have finished this gradient's encode pass
    unsigned char*      dense_scratch;
    double              base;
    uint32_t            G;
    uint32_t            tau;
    uint32_t            l;
};

// The launch arguments: up to kCmpMaxJobs gradients of the same length and parameters, compressed
// one after the other by the same resident grid (a block that is done with one gradient's encode
// pass starts summing the next while the others finish).
struct CmpBatch {
    const float*        grad[kCmpMaxJobs];
    uint8_t*            out[kCmpMaxJobs];
    uint64_t            out_bytes;
    uint64_t            n;
    Control*            ctl;
    double*             partials;        // [jobs][G]
    unsigned long long* desc;            // [jobs][G]
    unsigned long long* prefix;          // [jobs][G]
    float*              tmax;            // [jobs][G]
    uint32_t*           nelist;          // [jobs][G]
    uint32_t*           nebits;          // [jobs][ceil(G / 32)]
    unsigned int*       sm_slots;        // [256] blocks of this launch per SM
    unsigned char*      dense_scratch;
    double              base;
    uint32_t            jobs;
    uint32_t            G;
    uint32_t            tau;
    uint32_t            l;
    uint32_t            teams;           // 1, or 2: the two blocks of every SM work on different gradients
    uint32_t            pad;
    uint32_t            wait_limit;      // polls before a wait on another block gives up (kWaitLimit unless a test shortens it)
    uint32_t            try_limit;       // tries before a wait on a bulk copy gives up (kTryLimit likewise)
};

__device__ __forceinline__ CmpArgs job_view(const CmpBatch& b, uint32_t w) {
    CmpArgs a;
    a.grad = b.grad[w]; a.n = b.n; a.out = b.out[w]; a.out_bytes = b.out_bytes; a.ctl = b.ctl;
    a.ticket = b.ctl->tickets + w;
    a.partials = b.partials + (uint64_t)w * b.G;
    a.desc = b.desc + (uint64_t)w * b.G;
    a.prefix = b.prefix + (uint64_t)w * b.G;
    a.tmax = b.tmax + (uint64_t)w * b.G;
    a.nelist = b.nelist + (uint64_t)w * b.G;
    a.nebits = b.nebits + (uint64_t)w * ((b.G + 31u) >> 5);
    a.enc_done = b.ctl->enc_done + w;
    a.dense_scratch = b.dense_scratch; a.base = b.base; a.G = b.G; a.tau = b.tau; a.l = b.l;
    return a;
}

// ---- mbarrier / bulk-copy primitives (sm_90+ PTX) -------------------------------------------
__device__ __forceinline__ uint32_t smem_u32(const void* p) { return (uint32_t)__cvta_generic_to_shared(p); }
__device__ __forceinline__ void mbar_init(unsigned long long* bar, uint32_t count) {
    asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(smem_u32(bar)), "r"(count) : "memory");
}
__device__ __forceinline__ void mbar_expect_tx(unsigned long long* bar, uint32_t bytes) {
    asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(smem_u32(bar)), "r"(bytes) : "memory");
}
__device__ __forceinline__ void mbar_arrive(unsigned long long* bar) {
    asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(smem_u32(bar)) : "memory");
}
// Bounded wait: the hardware suspends the thread for up to about the hinted time per try, so a
// wait costs a handful of instructions; false when every try ran out.
constexpr uint32_t kTryHintNs = 10000u;
constexpr uint32_t kTryLimit  = 1u << 18;
__device__ __forceinline__ bool mbar_wait(unsigned long long* bar, uint32_t parity, uint32_t tries = kTryLimit) {
    const uint32_t addr = smem_u32(bar);
    for (uint32_t t = 0; t < tries; ++t) {
        uint32_t ok;
        asm volatile("{\n .reg .pred p;\n mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2, %3;\n selp.u32 %0, 1, 0, p;\n}"
                     : "=r"(ok) : "r"(addr), "r"(parity), "r"(kTryHintNs) : "memory");
        if (ok) return true;
    }
    return false;
}
__device__ __forceinline__ void bulk_load(void* dst_smem, const void* src_global, uint32_t bytes, unsigned long long* bar) {
    asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];"
                 ::"r"(smem_u32(dst_smem)), "l"(__cvta_generic_to_global(src_global)), "r"(bytes), "r"(smem_u32(bar))
                 : "memory");
}
// descriptors carry their whole payload in one word: relaxed accesses are enough
__device__ __forceinline__ unsigned long long ld_relaxed_u64(const unsigned long long* p) {
    unsigned long long v;
    asm volatile("ld.relaxed.gpu.global.u64 %0, [%1];" : "=l"(v) : "l"(p) : "memory");
    return v;
}
__device__ __forceinline__ void st_relaxed_u64(unsigned long long* p, unsigned long long v) {
    asm volatile("st.relaxed.gpu.global.u64 [%0], %1;" ::"l"(p), "l"(v) : "memory");
}
__device__ __forceinline__ void st_release_u32(unsigned int* p, unsigned int v) {
    asm volatile("st.release.gpu.global.u32 [%0], %1;" ::"l"(p), "r"(v) : "memory");
}
__device__ __forceinline__ unsigned int ld_acquire_u32(const unsigned int* p) {
    unsigned int v;
    asm volatile("ld.acquire.gpu.global.u32 %0, [%1];" : "=r"(v) : "l"(p) : "memory");
    return v;
}
// counter increment that publishes this thread's earlier writes and, for whoever comes last, makes the others' visible
__device__ __forceinline__ unsigned int atom_add_acq_rel_u32(unsigned int* p, unsigned int v) {
    unsigned int old;
    asm volatile("atom.acq_rel.gpu.global.add.u32 %0, [%1], %2;" : "=r"(old) : "l"(p), "r"(v) : "memory");
    return old;
}
// Phase stamps (%globaltimer, thread 0 of every block) are compiled in only with -DFASTSGD_TRACE.
#ifdef FASTSGD_TRACE
__device__ __forceinline__ unsigned long long read_globaltimer() {
    unsigned long long t;
    asm volatile("mov.u64 %0, %%globaltimer;" : "=l"(t));
    return t;
}
#define FSG_STAMP(slot) do { if (tid == 0) btrace[(slot)] = read_globaltimer(); } while (0)
#else
#define FSG_STAMP(slot) do { } while (0)
#endif

// Starts the copy of tile `tile` into `stage` (thread 0), and, for the one tile that reaches past
// n, fills the rest of the buffer (all threads).  Called by the whole block.
__device__ __forceinline__ void issue_tile(CmpSmem& s, const CmpArgs& a, int stage, uint32_t tile, int tid) {
    const uint64_t e0 = (uint64_t)tile << kGroupLog2;
    const uint64_t valid = min((uint64_t)kTile, a.n - e0);           // entries of this tile that exist
    const uint32_t bulk_bytes = (uint32_t)(valid * 4u) & ~15u;
    if (tid == 0) {
        if (bulk_bytes) {
            mbar_expect_tx(&s.mbar[stage], bulk_bytes);
            bulk_load(&s.stage[stage][0], a.grad + e0, bulk_bytes, &s.mbar[stage]);
        } else {
            mbar_arrive(&s.mbar[stage]);
        }
    }
    if (valid < kTile) {                                             // block-uniform
        for (uint32_t i = (bulk_bytes >> 2) + tid; i < kTile; i += kCmpThreads)
            s.stage[stage][i] = i < valid ? __ldg(a.grad + e0 + i) : 0.0f;
        __syncthreads();
        // these were generic-proxy writes to a buffer that a later bulk copy (async proxy) overwrites
        if (tid == 0) asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
    }
}

// Starts the copy of one part (kPartEntries entries) of a tile into its place in the stage, signalling mbar[part].
// Entries beyond n are zero (written by the threads themselves; block-wide call).
__device__ __forceinline__ void issue_part(CmpSmem& s, const CmpArgs& a, uint32_t tile, int part, int tid) {
    const uint64_t e0 = ((uint64_t)tile << kGroupLog2) + (uint64_t)part * kPartEntries;
    const uint64_t valid = e0 < a.n ? min((uint64_t)kPartEntries, a.n - e0) : 0ull;
    const uint32_t bulk_bytes = (uint32_t)(valid * 4u) & ~15u;
    float* dst = &s.stage[0][part * kPartEntries];
    if (tid == 0) {
        if (bulk_bytes) {
            mbar_expect_tx(&s.mbar[part], bulk_bytes);
            bulk_load(dst, a.grad + e0, bulk_bytes, &s.mbar[part]);
        } else {
            mbar_arrive(&s.mbar[part]);
        }
    }
    if (valid < kPartEntries) {                                      // block-uniform
        for (uint32_t i = (bulk_bytes >> 2) + tid; i < kPartEntries; i += kCmpThreads)
            dst[i] = i < valid ? __ldg(a.grad + e0 + i) : 0.0f;
        __syncthreads();
        // these were generic-proxy writes to a buffer that a later bulk copy (async proxy) overwrites
        if (tid == 0) asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
    }
}

// Tree node of the kPartRows rows of 128 entries a warp holds of a part (x[r]: this lane's 4 entries of row r).
__device__ __forceinline__ double warp_part_tree(const double (&x)[kPartRows], int lane) {
    if constexpr (kPartRows == 4) {
        return warp_halfslab_tree(reinterpret_cast<const double (&)[4]>(x), lane);
    } else {
        const bool b0 = lane & 1;
        const double keep = b0 ? x[1] : x[0], send = b0 ? x[0] : x[1];
        double u = __dadd_rn(keep, __shfl_xor_sync(kFullMask, send, 1));     // lanes 2k, 2k+1: 8 entries of row (lane & 1)
        u = __dadd_rn(u, __shfl_xor_sync(kFullMask, u, 2));                  // 16 entries
        u = __dadd_rn(u, __shfl_xor_sync(kFullMask, u, 4));                  // 32
        u = __dadd_rn(u, __shfl_xor_sync(kFullMask, u, 8));                  // 64
        u = __dadd_rn(u, __shfl_xor_sync(kFullMask, u, 16));                 // the row (128)
        u = __dadd_rn(u, __shfl_xor_sync(kFullMask, u, 1));                  // both rows = 256 entries
        return u;
    }
}

// Node of a whole tile from the parts' nodes of the 16 warps (s_warp[qp]) and its largest |v|; warp 0 only.
__device__ __forceinline__ void tile_node_from_parts(CmpSmem& s, const CmpArgs& a, uint32_t qp, uint32_t tile, int lane) {
    double t[kSumParts];
    uint32_t m = 0u;
#pragma unroll
    for (int p = 0; p < kSumParts; ++p) {
        t[p] = warp_tree(lane < kCmpWarps ? s.s_warp[qp][p][lane] : 0.0, kCmpWarps);
        m = max(m, lane < kCmpWarps ? s.s_wmax[qp][p][lane] : 0u);
    }
    const uint32_t tm = __reduce_max_sync(kFullMask, m);
    double node;
    if constexpr (kSumParts == 2) node = __dadd_rn(t[0], t[1]);
    else node = __dadd_rn(__dadd_rn(t[0], t[1]), __dadd_rn(t[2], t[3]));
    if (lane == 0) { a.partials[tile] = node; a.tmax[tile] = __uint_as_float(tm); }
}

// Tree reduction of the per-tile partials, by every block for itself, in passes of 512
// consecutive partials: thread t takes partial 512*p + t, the block forms that aligned node by
// shuffles (positions = lanes, then warps); the nodes of the passes are then reduced the same
// way.  Everything stays in registers and shared memory.
__device__ __forceinline__ double block_tree(double x, double* s_tree, int lane, int warp) {
    x = warp_tree(x);
    __syncthreads();                                   // s_tree may still be read from the last use
    if (lane == 0) s_tree[warp] = x;
    __syncthreads();
    double t = lane < kCmpWarps ? s_tree[lane] : 0.0;
    t = warp_tree(t, kCmpWarps);                       // lanes 0..15 of every warp hold the root
    return __shfl_sync(kFullMask, t, 0);
}

// BIG: with more than 8 passes a warp forms the node of a whole pass by itself (16 partials per lane,
// all in flight at once; the same tree by the transposing shuffle pattern) and the warps take the
// passes in turn.  (Only in the kernel variant for very many tiles: the tile loops of the others
// have proved sensitive to every bit of extra code around them.)
template <bool BIG>
__device__ __forceinline__ double reduce_partials(const double* partials, uint32_t chunks, double* s_tree,
                                                  double* s_nodes, int tid, int lane, int warp) {
    const uint32_t passes = (chunks + kCmpThreads - 1) / kCmpThreads;       // <= 256 for n < 2^31
    if (passes <= 8) {
        // thread t folds the aligned run of R = 1, 2, 4 or 8 partials that starts at R*t (all loads in
        // flight at once), then one tree over the threads: the same tree, one barrier pair
        const uint32_t R = passes <= 1 ? 1u : (passes <= 2 ? 2u : (passes <= 4 ? 4u : 8u));
        double v[8];
#pragma unroll
        for (int k = 0; k < 8; ++k) {
            const uint64_t idx = (uint64_t)tid * R + k;
            v[k] = ((uint32_t)k < R && idx < chunks) ? __ldcg(partials + idx) : 0.0;
        }
        // with R < 8 the unused slots are zero and x + 0 = x, so the full 8-leaf tree is still exact
        const double x = __dadd_rn(__dadd_rn(__dadd_rn(v[0], v[1]), __dadd_rn(v[2], v[3])),
                                   __dadd_rn(__dadd_rn(v[4], v[5]), __dadd_rn(v[6], v[7])));
        return block_tree(x, s_tree, lane, warp);
    }
    if constexpr (BIG) {
        for (uint32_t p = (uint32_t)warp; p < passes; p += kCmpWarps) {
            double x[16];
#pragma unroll
            for (int j = 0; j < 16; ++j) {
                const uint64_t idx = (uint64_t)p * kCmpThreads + 32u * (uint32_t)j + (uint32_t)lane;
                x[j] = idx < chunks ? __ldcg(partials + idx) : 0.0;
            }
            const double node = warp_rows16_tree(x, lane);
            if (lane == 0) s_nodes[p] = node;
        }
    } else {
    double next = (uint32_t)tid < chunks ? __ldcg(partials + tid) : 0.0;
    for (uint32_t p = 0; p < passes; ++p) {
        const double x = next;
        const uint64_t idx = (uint64_t)(p + 1) * kCmpThreads + tid;
        next = (p + 1 < passes && idx < chunks) ? __ldcg(partials + idx) : 0.0;    // in flight during this pass
        const double node = block_tree(x, s_tree, lane, warp);
        if (tid == 0) s_nodes[p] = node;
    }
    }
    __syncthreads();
    // the nodes of the passes, zero-padded to 512 positions, reduced on the same tree
    const double y = (uint32_t)tid < passes ? s_nodes[tid] : 0.0;
    return block_tree(y, s_tree, lane, warp);
}

// ceil(2^16 / M) for M = 1..20
__device__ __constant__ uint32_t c_inv_m[21] = {0, 65536, 32768, 21846, 16384, 13108, 10923, 9363, 8192, 7282, 6554, 5958,
                                                5462, 5042, 4682, 4370, 4096, 3856, 3641, 3450, 3277};

// flag of a delta with bit length bl: least f with ceil((f+1) M / 2^l) >= bl, which is
// floor((bl-1) 2^l / M) for bl >= 1; the division is a multiplication by ceil(2^16 / M)
__device__ __forceinline__ uint32_t flag_of(uint32_t delta, uint32_t l, uint32_t inv_m) {
    const uint32_t bl = delta ? 32u - __clz(delta) : 0u;
    return bl ? ((((bl - 1u) << l) * inv_m) >> 16) : 0u;
}

// L = least k in [0, tau] with |v| >= B_k (Eq. 2-3 as a table search; holds for k = tau), raised
// to 1, and the sign: the code byte.  The search starts from an estimate of log_b(S / |v|)
// (thr[130] = log2 S, thr[131] = 1 / log2 b, both approximate) and walks the non-increasing
// table from there, so the result does not depend on how good the estimate is.
__device__ __forceinline__ uint32_t code_byte_of(const float* thr, uint32_t tau, float val) {
    const float av = fabsf(val);
    int guess = (int)((thr[130] - __log2f(av)) * thr[131]) + 1;
    guess = max(0, min((int)tau, guess));
    uint32_t L = (uint32_t)guess;
    while (L > 0u && av >= thr[L - 1u]) --L;
    while (L < tau && av < thr[L]) ++L;
    L = L < 1u ? 1u : L;
    return (val < 0.0f ? 0x80u : 0u) | (L - 1u);
}

// Phase 2 for a tile too dense for the per-warp lists.  The kept (key, value) pairs are compacted
// in index order into the block's slot of global scratch (coalesced, L2-resident); the stage, whose
// values are dead after that, then holds the blob (at most 16384 x 27 bits): code bytes by plain
// byte stores, then flags and deltas 512 keys at a time (one block-wide scan of the widths per
// chunk) with shared-memory ORs.  The caller places the blob from the stage before it refills it.
// `m` is the kept mask of this thread's 32 entries.
static_assert((uint64_t)kTile * (8u + 5u + (uint32_t)kGroupLog2) <= (uint64_t)kTile * 32u, "the widest blob fits the stage");

// (A real call, with plain values only: the sparse workloads' tile loop stays small.)  Returns words | M << 32.
__device__ __noinline__ unsigned long long pack_tile_dense(CmpSmem* sp, unsigned char* dense_scratch, uint32_t a_l, uint32_t a_tau,
                                                           uint32_t count, uint32_t warp_base, uint32_t m,
                                                           uint32_t ex0, uint32_t ex1, uint32_t tot0, uint32_t tot1) {
    CmpSmem& s = *sp;
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    unsigned char* slot = dense_scratch + (uint64_t)blockIdx.x * kDenseScratchBytes;
    uint32_t* vals = reinterpret_cast<uint32_t*>(slot);
    uint16_t* keys = reinterpret_cast<uint16_t*>(slot + (uint64_t)kTile * 4u);
    const float* tile = s.stage[0];
    uint32_t* blob = reinterpret_cast<uint32_t*>(s.stage[0]);

    // ---- stream compaction in index order: (key, value) of the kept entries
    if (m != 0u) {
        uint32_t row_base = warp_base;
#pragma unroll
        for (int r = 0; r < 8; ++r) {
            const uint32_t tot = r < 4 ? (tot0 >> (8 * r)) & 0xFFu : (tot1 >> (8 * (r - 4))) & 0xFFu;
            const uint32_t ex  = r < 4 ? (ex0 >> (8 * r)) & 0xFFu : (ex1 >> (8 * (r - 4))) & 0xFFu;
            const uint32_t mr = (m >> (4 * r)) & 0xFu;
            uint32_t pos = row_base + ex;
            const uint32_t k0 = warp * 1024 + r * 128 + lane * 4;
            if (mr) {
                if (mr & 1u) { keys[pos] = (uint16_t)(k0);     vals[pos] = __float_as_uint(tile[k0]);     ++pos; }
                if (mr & 2u) { keys[pos] = (uint16_t)(k0 + 1); vals[pos] = __float_as_uint(tile[k0 + 1]); ++pos; }
                if (mr & 4u) { keys[pos] = (uint16_t)(k0 + 2); vals[pos] = __float_as_uint(tile[k0 + 2]); ++pos; }
                if (mr & 8u) { keys[pos] = (uint16_t)(k0 + 3); vals[pos] = __float_as_uint(tile[k0 + 3]); ++pos; }
            }
            row_base += tot;
        }
    }
    if (tid == 0) s.max_delta = 0u;
    __syncthreads();                          // the stage's values are dead from here on

    // ---- zero the words the blob can reach
    {
        const uint32_t bound_words = (count * (8u + a_l + (uint32_t)kGroupLog2) + 31u) >> 5;
        for (uint32_t i = tid; i < bound_words; i += kCmpThreads) blob[i] = 0u;
    }
    __syncthreads();

    // ---- logarithm quantisation (code bytes straight to their place: byte j of the stream is the
    //      byte 3 - j%4 of big-endian-valued word j/4) and the largest delta (Eq. 4)
    {
        uint8_t* blob_bytes = reinterpret_cast<uint8_t*>(blob);
        uint32_t local_max = 0;
        for (uint32_t j = tid; j < count; j += kCmpThreads) {
            const uint32_t key = keys[j];
            const uint32_t prev = j ? (uint32_t)keys[j - 1] : 0u;      // (the first delta of a group counts from 0)
            blob_bytes[(j & ~3u) | (3u - (j & 3u))] = (uint8_t)code_byte_of(s.thr, a_tau, __uint_as_float(vals[j]));
            local_max = max(local_max, key - prev);
        }
        local_max = __reduce_max_sync(kFullMask, local_max);
        if (lane == 0 && local_max) atomicMax(&s.max_delta, local_max);
    }
    __syncthreads();

    // ---- M; flags and deltas, 512 consecutive keys per round
    const uint32_t maxd = s.max_delta;
    const uint32_t M = maxd ? (32u - __clz(maxd)) : 1u;
    const uint32_t inv_m = c_inv_m[M];
    const uint32_t round_up = (1u << a_l) - 1u;
    const uint32_t flag_pos0 = 8u * count, delta_pos0 = flag_pos0 + a_l * count;
    uint32_t dbase = delta_pos0;
    for (uint32_t j0 = 0, round = 0; j0 < count; j0 += kCmpThreads, ++round) {
        const uint32_t j = j0 + (uint32_t)tid;
        uint32_t delta = 0, f = 0, w = 0;
        if (j < count) {
            delta = (uint32_t)keys[j] - (j ? (uint32_t)keys[j - 1] : 0u);
            f = flag_of(delta, a_l, inv_m);
            w = ((f + 1u) * M + round_up) >> a_l;
        }
        const uint32_t incl = warp_incl_scan(w, lane);
        if (lane == 31) s.scan_tot2[round & 1u][warp] = incl;
        __syncthreads();                      // (one barrier per round: the totals are double-buffered)
        uint32_t before = 0, all = 0;
#pragma unroll
        for (int k = 0; k < kCmpWarps; ++k) {
            const uint32_t t = s.scan_tot2[round & 1u][k];
            if (k < warp) before += t;
            all += t;
        }
        if (j < count) {
            put_bits_smem(blob, flag_pos0 + a_l * j, f, a_l);
            put_bits_smem(blob, dbase + before + (incl - w), delta, w);
        }
        dbase += all;
    }
    __syncthreads();      // blob complete
    return (unsigned long long)((dbase + 31u) >> 5) | ((unsigned long long)M << 32);
}

// Running exclusive scan of the descriptors, kept by every block for itself.
struct ScanState {
    uint32_t pos;          // descriptors [0, pos) are included
    uint32_t count;        // kept entries in groups [0, pos)
    uint32_t words;        // blob words of groups [0, pos)
};

// Copies the blobs of the pending tiles [pbeg, npend) of one gradient to their places in the stream
// (pend_prefix holds each tile's exclusive prefix), writes their directory entries and, for the
// last group, the header.  No barrier inside.
__device__ __forceinline__ void place_pending(CmpSmem& s, const CmpArgs& a, uint32_t jp, int pbeg, int npend, int tid, int lane, int warp) {
    const double S = s.job_sum[jp];
    const uint32_t skip = s.job_skip[jp];
    // ---- copy-out, directory entries, header
    const uint32_t fixed_words = (kHeaderBytes + 8u * a.G) >> 2;
    uint32_t* outw = reinterpret_cast<uint32_t*>(a.out);
    // one warp per pending tile (a dense tile's blob, in global scratch, is copied by the whole block)
    for (int p0 = pbeg; p0 < npend; p0 += kCmpWarps) {
        const int p = p0 + warp;
        const bool mine = p < npend;
        const uint32_t g = mine ? s.pend_g[p] : 0u, cm = mine ? s.pend_cm[p] : 0u, words = mine ? s.pend_words[p] : 0u,
                       aoff = mine ? s.pend_off[p] : 0u;
        const unsigned long long pre = mine ? s.pend_prefix[p] : 0ull;
        const uint32_t off = fixed_words + (uint32_t)pre;
        const uint64_t end_bytes = ((uint64_t)off + words) << 2;
        if (mine && aoff != kDenseMark && end_bytes <= a.out_bytes) {
            const uint32_t* blob = s.arena + aoff;
            for (uint32_t i = lane; i < words; i += 32) outw[off + i] = bswap32(blob[i]);
        }
        if (mine && lane == 0) {
            outw[(kHeaderBytes >> 2) + 2 * g]     = cm;
            outw[(kHeaderBytes >> 2) + 2 * g + 1] = off;
        }
        if (mine && g == a.G - 1 && lane == 0) {
            int status = kStOk;
            if (ld_acquire_u32(&a.ctl->error) != 0u) status = kStTimeout;      // some block of the launch gave up: its tiles are missing
            else if (skip == 2u) status = kStNonfinite;
            else if (end_bytes > a.out_bytes) status = kStCapacity;
            const uint64_t d_total = status == kStOk ? (pre >> 32) + (cm & 0xFFFFFFu) : 0ull;
            const uint64_t total = status == kStOk ? end_bytes : (uint64_t)kHeaderBytes;
            const double Sh = (status == kStNonfinite || status == kStTimeout) ? 0.0 : S;
            outw[0] = kMagic;
            outw[1] = kVersion;
            outw[2] = (uint32_t)status;
            outw[3] = a.tau;
            outw[4] = (uint32_t)a.n;            outw[5] = (uint32_t)(a.n >> 32);
            outw[6] = (uint32_t)d_total;        outw[7] = (uint32_t)(d_total >> 32);
            outw[8] = (uint32_t)total;          outw[9] = (uint32_t)(total >> 32);
            const unsigned long long sb = (unsigned long long)__double_as_longlong(Sh);
            const unsigned long long bb = (unsigned long long)__double_as_longlong(a.base);
            outw[10] = (uint32_t)sb;            outw[11] = (uint32_t)(sb >> 32);
            outw[12] = (uint32_t)bb;            outw[13] = (uint32_t)(bb >> 32);
            outw[14] = a.l | ((uint32_t)kGroupLog2 << 8);
            outw[15] = a.G;
        }
    }
    // the blob of a tile that took the dense path (at most one is pending) waits in the block's slot of global scratch
    for (int p = pbeg; p < npend; ++p) {
        if (s.pend_off[p] != kDenseMark) continue;
        const uint32_t words = s.pend_words[p];
        const uint32_t off = fixed_words + (uint32_t)s.pend_prefix[p];
        const uint64_t end_bytes = ((uint64_t)off + words) << 2;
        const uint32_t* blob = reinterpret_cast<const uint32_t*>(a.dense_scratch + (uint64_t)blockIdx.x * kDenseScratchBytes);
        if (end_bytes <= a.out_bytes)
            for (uint32_t i = tid; i < words; i += kCmpThreads) outw[off + i] = bswap32(__ldcg(blob + i));
    }
}

// Pending tiles [0, n) belong to a gradient whose encode pass is over or nearly so: the last block
// to finish it writes the exclusive scan of all its descriptors (publish_prefixes).  Fetches the
// entries of these tiles (bounded polls); a failure shows in s.poison_seen after the next barrier.
__device__ __forceinline__ void fetch_prefixes(CmpSmem& s, const CmpArgs& a, int n, int tid) {
    if (tid < n) {
        const unsigned long long* p = a.prefix + s.pend_g[tid];
        unsigned long long v = ld_relaxed_u64(p);
        uint32_t spin = 0;
        while ((v >> 62) == kDescInvalid) {
            if (++spin > s.wait_limit) { s.poison_seen = 2u; break; }
            if (spin > 32u) __nanosleep(32);
            v = ld_relaxed_u64(p);
        }
        if ((v >> 62) == kDescPoison) s.poison_seen = 1u;
        s.pend_prefix[tid] = ((unsigned long long)desc_count(v) << 32) | desc_words(v);
    }
}

// Gives every pending tile its place in the stream and empties the arena.  Tiles [0, nprev) of the
// list belong to the previous gradient (view ap, slot jp ^ 1): their prefixes come from the
// published scan.  Tiles [nprev, npend) belong to the gradient being encoded (view a, slot jp;
// group numbers ascend): the block advances its own scan of the descriptors up to them.  Returns
// false if a poisoned descriptor or a timeout was met (the caller aborts).
// First half (drain_wait): everything that may have to wait for other blocks; when it returns every
// pending tile's prefix is known.  Second half (drain_place): the copies.
__device__ __forceinline__ bool drain_wait(CmpSmem& s, const CmpArgs& a, const CmpArgs& ap, int nprev, int npend,
                                           int tid, int lane, int warp) {
    if (tid == 0) s.poison_seen = 0u;
    __syncthreads();
    fetch_prefixes(s, ap, nprev, tid);
    if (npend == nprev) {
        __syncthreads();
        return s.poison_seen == 0u;        // (rewritten only at the start of the next drain, behind a barrier)
    }
    ScanState sc; sc.pos = s.sc_pos; sc.count = s.sc_count; sc.words = s.sc_words;
    const uint32_t g_last = s.pend_g[npend - 1];
    // ---- advance the scan over descriptors [sc.pos, g_last]: batches of kDrainChunks x 512, all loads
    //      of a batch in flight at once, one shuffle scan per chunk, two barriers per batch
    while (sc.pos <= g_last) {
        unsigned long long own[kDrainChunks], excl[kDrainChunks];
#pragma unroll
        for (int j = 0; j < kDrainChunks; ++j) {
            const uint32_t idx = sc.pos + (uint32_t)j * kCmpThreads + tid;
            own[j] = idx <= g_last ? ld_relaxed_u64(a.desc + idx) : desc_pack(kDescValid, 0, 0);
        }
#pragma unroll
        for (int j = 0; j < kDrainChunks; ++j) {
            const uint32_t idx = sc.pos + (uint32_t)j * kCmpThreads + tid;
            uint32_t spin = 0;
            while ((own[j] >> 62) == kDescInvalid) {         // not published yet: bounded poll
                if (++spin > s.wait_limit) { s.poison_seen = 2u; own[j] = 0ull; break; }
                __nanosleep(64);
                own[j] = ld_relaxed_u64(a.desc + idx);
            }
            if ((own[j] >> 62) == kDescPoison) { s.poison_seen = 1u; own[j] = 0ull; }
            own[j] = ((unsigned long long)desc_count(own[j]) << 32) | desc_words(own[j]);
            unsigned long long incl = own[j];
#pragma unroll
            for (int o = 1; o < 32; o <<= 1) {
                const unsigned long long t = __shfl_up_sync(kFullMask, incl, o);
                if (lane >= o) incl += t;
            }
            if (lane == 31) s.scan64[j][warp] = incl;
            excl[j] = incl - own[j];
        }
        __syncthreads();
        unsigned long long running = ((unsigned long long)sc.count << 32) | sc.words;
#pragma unroll
        for (int j = 0; j < kDrainChunks; ++j) {
            unsigned long long before = running, all = 0ull;
#pragma unroll
            for (int w = 0; w < kCmpWarps; ++w) {
                const unsigned long long t = s.scan64[j][w];
                if (w < warp) before += t;
                all += t;
            }
            excl[j] += before;                               // exclusive prefix of descriptor sc.pos + 512 j + tid
            running += all;
        }
        // the thread that holds one of this block's pending tiles records that tile's exclusive prefix
        for (int p = nprev; p < npend; ++p) {
            const uint32_t idx = s.pend_g[p];
            if (idx < sc.pos || idx >= sc.pos + (uint32_t)kDrainChunks * kCmpThreads) continue;
            const uint32_t rel = idx - sc.pos;
            if ((rel % kCmpThreads) != (uint32_t)tid) continue;
            const int jj = (int)(rel / kCmpThreads);
            unsigned long long e = 0ull;
#pragma unroll
            for (int j = 0; j < kDrainChunks; ++j) if (j == jj) e = excl[j];
            s.pend_prefix[p] = e;
        }
        sc.count = (uint32_t)(running >> 32);
        sc.words = (uint32_t)running;
        sc.pos += (uint32_t)kDrainChunks * kCmpThreads;
        const uint32_t poison_now = s.poison_seen;      // read between the barriers: same value in every thread
        __syncthreads();
        if (poison_now) return false;
    }
    // the scan ran past g_last by whole steps: pull it back to g_last + 1
    // (descriptors beyond g_last were read as zero, so only the position needs correcting)
    sc.pos = g_last + 1u;
    if (tid == 0) { s.sc_pos = sc.pos; s.sc_count = sc.count; s.sc_words = sc.words; }   // (read again after a later barrier)
    return true;
}

__device__ __forceinline__ void drain_place(CmpSmem& s, const CmpArgs& a, const CmpArgs& ap, uint32_t jp, int nprev, int npend,
                                            int tid, int lane, int warp) {
    place_pending(s, ap, jp ^ 1u, 0, nprev, tid, lane, warp);
    place_pending(s, a, jp, nprev, npend, tid, lane, warp);
    __syncthreads();                       // the arena and the pending list are free again
}

__device__ __forceinline__ bool drain(CmpSmem& s, const CmpArgs& a, const CmpArgs& ap, uint32_t jp, int nprev, int npend,
                                      int tid, int lane, int warp) {
    if (npend == 0) return true;
    if (!drain_wait(s, a, ap, nprev, npend, tid, lane, warp)) return false;
    drain_place(s, a, ap, jp, nprev, npend, tid, lane, warp);
    return true;
}

// Places tiles [0, n) of the list, all of one gradient whose encode pass is over (slot jp).
__device__ __forceinline__ bool drain_final(CmpSmem& s, const CmpArgs& a, uint32_t jp, int n, int tid, int lane, int warp) {
    if (n == 0) return true;
    if (tid == 0) s.poison_seen = 0u;
    __syncthreads();
    fetch_prefixes(s, a, n, tid);
    __syncthreads();
    if (s.poison_seen) return false;       // (rewritten only at the start of the next drain, behind a barrier)
    place_pending(s, a, jp, 0, n, tid, lane, warp);
    __syncthreads();
    return true;
}

// Exclusive scan of all descriptors of a gradient into a.prefix, kDrainChunks x 512 at a time.
// POLL = false: run by the last block to finish the gradient's encode pass (every descriptor is
// published by then).  POLL = true: run by the first block to finish it, which follows the
// others' descriptors as they appear (bounded polls), so that the prefixes are complete right
// after the last tile is published -- used for the launch's last gradient, where everybody waits
// for them.  A descriptor that is not valid (or never comes) poisons its own and every later prefix.
template <bool POLL, int kChunks>
__device__ __forceinline__ void publish_prefixes(CmpSmem& s, const CmpArgs& a, int tid, int lane, int warp) {
    const uint32_t fixed_words = (kHeaderBytes + 8u * a.G) >> 2;
    uint32_t* outw = reinterpret_cast<uint32_t*>(a.out);
    unsigned long long running = 0ull;
    bool bad = false;
    for (uint32_t pos = 0; pos < a.G; pos += (uint32_t)kChunks * kCmpThreads) {
        unsigned long long own[kChunks], excl[kChunks];
        bool bad_here = false;
#pragma unroll
        for (int j = 0; j < kChunks; ++j) {
            const uint32_t idx = pos + (uint32_t)j * kCmpThreads + tid;
            own[j] = idx < a.G ? ld_relaxed_u64(a.desc + idx) : desc_pack(kDescValid, 0, 0);
        }
#pragma unroll
        for (int j = 0; j < kChunks; ++j) {
            if (POLL && !bad) {
                const uint32_t idx = pos + (uint32_t)j * kCmpThreads + tid;
                uint32_t spin = 0;
                while ((own[j] >> 62) == kDescInvalid) {         // not published yet: bounded poll
                    if (++spin > s.wait_limit) break;
                    if (spin > 32u) __nanosleep(32);
                    own[j] = ld_relaxed_u64(a.desc + idx);
                }
            }
            if ((own[j] >> 62) != kDescValid) { bad_here = true; own[j] = 0ull; }
            own[j] = ((unsigned long long)desc_count(own[j]) << 32) | desc_words(own[j]);
            unsigned long long incl = own[j];
#pragma unroll
            for (int o = 1; o < 32; o <<= 1) {
                const unsigned long long t = __shfl_up_sync(kFullMask, incl, o);
                if (lane >= o) incl += t;
            }
            if (lane == 31) s.scan64[j][warp] = incl;
            excl[j] = incl - own[j];
        }
        if (__syncthreads_or(bad_here ? 1 : 0)) bad = true;
#pragma unroll
        for (int j = 0; j < kChunks; ++j) {
            unsigned long long before = running, all = 0ull;
#pragma unroll
            for (int w = 0; w < kCmpWarps; ++w) {
                const unsigned long long t = s.scan64[j][w];
                if (w < warp) before += t;
                all += t;
            }
            excl[j] += before;
            running += all;
            const uint32_t idx = pos + (uint32_t)j * kCmpThreads + tid;
            if (idx < a.G) {
                st_relaxed_u64(a.prefix + idx, bad ? desc_pack(kDescPoison, 0, 0)
                                                   : desc_pack(kDescValid, (uint32_t)(excl[j] >> 32), (uint32_t)excl[j]));
                // a group without kept entries: its directory entry (most of these tiles were never read by the encode pass)
                if (!bad && (own[j] >> 32) == 0ull) {
                    outw[(kHeaderBytes >> 2) + 2u * idx]      = 0u;
                    outw[(kHeaderBytes >> 2) + 2u * idx + 1u] = fixed_words + (uint32_t)excl[j];
                }
            }
        }
        __syncthreads();
    }
}

// The same scan shared among the first blocks to finish the encode pass (kernel variant for very many tiles:
// one block scanning 16384 descriptors or more takes tens of microseconds at the very end of the launch).
// Block number `part` of `parts` takes a contiguous segment of the descriptors: it adds the segment up,
// following descriptors that are not published yet (bounded polls), publishes the segment's total, takes
// the totals of the segments before it (published the same way: bounded polls; nobody waits for a later
// segment, so there is no cycle), then scans its segment once more from that base and writes the prefixes
// and the directory entries of the groups without kept entries.  A descriptor that is not valid poisons
// the prefixes of its segment and of every later one.
constexpr uint32_t kScanParts = 16;
__device__ __forceinline__ unsigned long long scan_segment(CmpSmem& s, const CmpArgs& a, uint32_t beg, uint32_t end, unsigned long long running,
                                                          bool store, bool& bad, int tid, int lane, int warp) {
    const uint32_t fixed_words = (kHeaderBytes + 8u * a.G) >> 2;
    uint32_t* outw = reinterpret_cast<uint32_t*>(a.out);
    for (uint32_t pos = beg; pos < end; pos += (uint32_t)kDrainChunks * kCmpThreads) {
        unsigned long long own[kDrainChunks], excl[kDrainChunks];
        bool bad_here = false;
#pragma unroll
        for (int j = 0; j < kDrainChunks; ++j) {
            const uint32_t idx = pos + (uint32_t)j * kCmpThreads + tid;
            own[j] = idx < end ? ld_relaxed_u64(a.desc + idx) : desc_pack(kDescValid, 0, 0);
        }
#pragma unroll
        for (int j = 0; j < kDrainChunks; ++j) {
            if (!store && !bad) {
                const uint32_t idx = pos + (uint32_t)j * kCmpThreads + tid;
                uint32_t spin = 0;
                while ((own[j] >> 62) == kDescInvalid) {         // not published yet: bounded poll
                    if (++spin > s.wait_limit) break;
                    if (spin > 32u) __nanosleep(32);
                    own[j] = ld_relaxed_u64(a.desc + idx);
                }
            }
            if ((own[j] >> 62) != kDescValid) { bad_here = true; own[j] = 0ull; }
            own[j] = ((unsigned long long)desc_count(own[j]) << 32) | desc_words(own[j]);
            unsigned long long incl = own[j];
#pragma unroll
            for (int o = 1; o < 32; o <<= 1) {
                const unsigned long long u = __shfl_up_sync(kFullMask, incl, o);
                if (lane >= o) incl += u;
            }
            if (lane == 31) s.scan64[j][warp] = incl;
            excl[j] = incl - own[j];
        }
        if (__syncthreads_or(bad_here ? 1 : 0)) bad = true;
#pragma unroll
        for (int j = 0; j < kDrainChunks; ++j) {
            unsigned long long before = running, all = 0ull;
#pragma unroll
            for (int w = 0; w < kCmpWarps; ++w) {
                const unsigned long long u = s.scan64[j][w];
                if (w < warp) before += u;
                all += u;
            }
            excl[j] += before;
            running += all;
            const uint32_t idx = pos + (uint32_t)j * kCmpThreads + tid;
            if (store && idx < end) {
                st_relaxed_u64(a.prefix + idx, bad ? desc_pack(kDescPoison, 0, 0)
                                                   : desc_pack(kDescValid, (uint32_t)(excl[j] >> 32), (uint32_t)excl[j]));
                if (!bad && (own[j] >> 32) == 0ull) {
                    outw[(kHeaderBytes >> 2) + 2u * idx]      = 0u;
                    outw[(kHeaderBytes >> 2) + 2u * idx + 1u] = fixed_words + (uint32_t)excl[j];
                }
            }
        }
        __syncthreads();
    }
    return running;
}

__device__ __forceinline__ void publish_part(CmpSmem& s, const CmpArgs& a, unsigned long long* segtot, uint32_t part, uint32_t parts,
                                             int tid, int lane, int warp) {
    constexpr uint32_t kStepAll = (uint32_t)kDrainChunks * kCmpThreads;
    const uint32_t seg = ((a.G + parts - 1u) / parts + kStepAll - 1u) / kStepAll * kStepAll;
    const uint32_t beg = min(part * seg, a.G), end = min(beg + seg, a.G);
    bool bad = false;
    const unsigned long long total = scan_segment(s, a, beg, end, 0ull, false, bad, tid, lane, warp);
    if (tid == 0) st_relaxed_u64(segtot + part, bad ? desc_pack(kDescPoison, 0, 0) : desc_pack(kDescValid, (uint32_t)(total >> 32), (uint32_t)total));
    // the segments before this one
    if (tid < (int)kScanParts) s.scan64[0][tid] = 0ull;
    if (tid == 0) s.pad5 = 0u;                          // (set below if one of them is poisoned)
    __syncthreads();
    if (tid < (int)part) {
        unsigned long long v = ld_relaxed_u64(segtot + tid);
        uint32_t spin = 0;
        while ((v >> 62) == kDescInvalid) {
            if (++spin > s.wait_limit) break;
            if (spin > 32u) __nanosleep(32);
            v = ld_relaxed_u64(segtot + tid);
        }
        if ((v >> 62) != kDescValid) s.pad5 = 1u;
        s.scan64[0][tid] = ((unsigned long long)desc_count(v) << 32) | desc_words(v);
    }
    __syncthreads();
    unsigned long long base = 0ull;
#pragma unroll
    for (int w = 0; w < (int)kScanParts; ++w) base += s.scan64[0][w];
    if (s.pad5) bad = true;
    __syncthreads();
    scan_segment(s, a, beg, end, base, true, bad, tid, lane, warp);
}

// Every stream of the launch reports the timeout: a header with that status and nothing else (identical words from
// every block that writes them).  One thread.
__device__ __forceinline__ void write_timeout_headers(const CmpBatch& b) {
    for (uint32_t w = 0; w < b.jobs; ++w) {
        uint32_t* outw = reinterpret_cast<uint32_t*>(b.out[w]);
        outw[0] = kMagic; outw[1] = kVersion; outw[2] = (uint32_t)kStTimeout; outw[3] = b.tau;
        outw[4] = (uint32_t)b.n; outw[5] = (uint32_t)(b.n >> 32);
        outw[6] = 0u; outw[7] = 0u; outw[8] = kHeaderBytes; outw[9] = 0u;
        outw[10] = 0u; outw[11] = 0u;
        const unsigned long long bb = (unsigned long long)__double_as_longlong(b.base);
        outw[12] = (uint32_t)bb; outw[13] = (uint32_t)(bb >> 32);
        outw[14] = b.l | ((uint32_t)kGroupLog2 << 8);
        outw[15] = b.G;
    }
}

// Phase 1 for one gradient: fp64 partial sum of every 2^14-entry tile.  Tiles grid..G-1 are handed
// out by a ticket counter (so that the blocks finish together; with one gradient from the last
// tile down, so that the encode pass starts on what L2 still holds); the block's own tile c comes
// last (and stays in the stage afterwards).  Thread 0 holds the ticket of the tile after the one at
// hand, taken one iteration before it is used.  sum_begin starts the copy of the first tile and
// returns; sum_rest does the rest (the caller has something else to do while that copy flies).
// `limit` bounds the tiles the block takes (a block that only helps with a pass).
struct SumCursor {
    unsigned int tk;       // thread 0: the look-ahead ticket
    uint32_t     tile;     // the tile whose copy is in flight
};

__device__ __forceinline__ SumCursor sum_begin(CmpSmem& s, const CmpArgs& a, uint32_t job, bool full, uint32_t c, uint32_t grid,
                                               uint32_t limit, uint32_t& pending, int tid) {
    SumCursor cur; cur.tk = 0u;
    if (tid == 0) {
        cur.tk = atomicAdd(a.ctl->tickets1 + job, 1u);
        s.p1_next[0] = full ? (cur.tk < a.G ? cur.tk : kNoTicket) : (grid + cur.tk < a.G ? a.G - 1u - cur.tk : c);
    }
    __syncthreads();
    cur.tile = s.p1_next[0];
    if (cur.tile != kNoTicket) {
#pragma unroll
        for (int part = 0; part < kSumParts; ++part) issue_part(s, a, cur.tile, part, tid);
        pending |= (1u << kSumParts) - 1u;
        if (tid == 0 && limit > 1u && (full || cur.tile != c)) cur.tk = atomicAdd(a.ctl->tickets1 + job, 1u);
    }
    return cur;
}

// The tile goes through the stage in kSumParts parts with a barrier each: as soon as the block has read
// a part it starts the copy of the same part of its next tile, so that all the other parts' copies are in
// flight while one part is being summed (with two blocks per SM the bytes in flight, not the arithmetic,
// bound this pass).  Warp w sums the w-th sixteenth of the part; the tile's node is the tree over its
// parts' nodes (the same fixed tree as everywhere).
__device__ __forceinline__ void sum_rest(CmpSmem& s, const CmpArgs& a, uint32_t job, bool full, uint32_t c, uint32_t grid,
                                         uint32_t limit, SumCursor cur, uint32_t& parity, uint32_t& pending,
                                         int tid, int lane, int warp) {
    unsigned int tk = cur.tk;
    uint32_t tile = cur.tile;
    if (tile == kNoTicket) return;                    // (several gradients, fewer tiles than blocks)
    uint32_t prev_tile = kNoTicket;                   // its halves' nodes wait in s_warp[(q - 1) & 1]
    uint32_t q = 0;
    for (;; ++q) {
        const uint32_t qp = q & 1u;
        if (tid == 0) {
            a.desc[tile] = 0ull; a.prefix[tile] = 0ull;   // phase 2's descriptors and prefixes (ordered by the grid barrier)
            // the tile after this one: a ticketed tile, then (one gradient) c, then none
            s.p1_next[(q + 1) & 1] = q + 1u >= limit ? kNoTicket
                                     : full ? (tk < a.G ? tk : kNoTicket)
                                            : (tile == c ? kNoTicket : (grid + tk < a.G ? a.G - 1u - tk : c));
        }
        uint32_t nxt = kNoTicket;
#pragma unroll
        for (int part = 0; part < kSumParts; ++part) {
            if (!mbar_wait(&s.mbar[part], (parity >> part) & 1u, s.try_limit)) s.abort_flag = 1u;
            parity ^= 1u << part;
            pending &= ~(1u << part);
            double x[kPartRows];
            float mx = 0.0f;
            const float4* row = reinterpret_cast<const float4*>(&s.stage[0][part * (int)kPartEntries + warp * (int)(kPartEntries / kCmpWarps)]) + lane;
#pragma unroll
            for (int r = 0; r < kPartRows; ++r) {
                const float4 v4 = row[r * 32];
                x[r] = abs_sum4(v4);
                mx = fmaxf(mx, fmaxf(fmaxf(fabsf(v4.x), fabsf(v4.y)), fmaxf(fabsf(v4.z), fabsf(v4.w))));
            }
            __syncthreads();                          // the part has been read (and p1_next is visible)
            if (s.abort_flag) return;
            if (part == 0) nxt = s.p1_next[(q + 1) & 1];
            if (nxt != kNoTicket) {                   // (with one gradient the last tile, c, stays in the stage)
                issue_part(s, a, nxt, part, tid);
                pending |= 1u << part;
            }
            const double u = warp_part_tree(x, lane);
            const uint32_t wmx = __reduce_max_sync(kFullMask, __float_as_uint(mx));     // (non-negative floats order like their bits; a NaN shows in the sum)
            if (lane == 0) { s.s_warp[qp][part][warp] = u; s.s_wmax[qp][part][warp] = wmx; }
            // the tile before this one: all of its parts' nodes are complete since the barrier above
            if (part == 0 && warp == 0 && prev_tile != kNoTicket) tile_node_from_parts(s, a, qp ^ 1u, prev_tile, lane);
        }
        prev_tile = tile;
        if (nxt == kNoTicket) break;
        if (tid == 0 && q + 2u < limit && (full || nxt != c)) tk = atomicAdd(a.ctl->tickets1 + job, 1u);
        tile = nxt;
    }
    // the last tile's nodes
    __syncthreads();
    if (warp == 0) tile_node_from_parts(s, a, q & 1u, prev_tile, lane);
}

// Run by one block when a gradient's sum S is known: which tiles does the encode pass have to read?
// A tile whose largest |v| (recorded by the sum pass) is below the early-stop threshold B_tau holds
// nothing to keep.  Such a tile gets its descriptor (0 entries, 0 words) here; its directory entry
// is written by the block that publishes the prefixes.  The others go into a.nelist in ascending
// order, and the encode pass hands out positions of that list.  Tiles below first_ticketed are not
// listed (with one gradient each block encodes its own tile, which it still holds); the last tile
// is always listed, since whoever encodes it writes the header.  Returns the length of the list
// (valid in thread 0).
// The first kListAhead x 512 tiles' maxima, asked for before the partials are reduced (the two waits overlap).
constexpr int kListAhead = 8;
__device__ __forceinline__ void tile_maxima_ahead(const CmpArgs& a, float (&tm)[kListAhead], int tid) {
#pragma unroll
    for (int j = 0; j < kListAhead; ++j) {
        const uint32_t tile = (uint32_t)j * kCmpThreads + tid;
        tm[j] = tile < a.G ? __ldcg(a.tmax + tile) : 0.0f;
    }
}

template <bool BIG>
__device__ __forceinline__ uint32_t build_tile_list(CmpSmem& s, const CmpArgs& a, const PowTable& pw, double S, uint32_t first_ticketed,
                                                    const float (&tm_ahead)[kListAhead], int tid, int lane, int warp) {
    // the threshold exactly as the encode pass forms it
    const float thr_e = isfinite(S) ? fmaxf(__double2float_ru(__ddiv_rn(S, pw.P[a.tau])), __int_as_float(1)) : __int_as_float(0x7f800000);
    constexpr int kInFlight = BIG ? 16 : kListAhead;
    // the bitmap of the listed tiles: in shared memory (the scratch of the partials' reduction, free by now) unless the
    // gradient has very many tiles
    const bool bits_global = BIG || a.G > 8u * (uint32_t)sizeof(s.s_nodes);
    uint32_t* bits = bits_global ? a.nebits : reinterpret_cast<uint32_t*>(s.s_nodes);
    for (uint32_t base = 0; base < a.G; base += (uint32_t)kInFlight * kCmpThreads) {
        float tm[kInFlight];
#pragma unroll
        for (int j = 0; j < kInFlight; ++j) {
            const uint32_t tile = base + (uint32_t)j * kCmpThreads + tid;
            if (!BIG && base == 0u) tm[j] = tm_ahead[j < kListAhead ? j : 0];
            else tm[j] = tile < a.G ? __ldcg(a.tmax + tile) : 0.0f;
        }
#pragma unroll
        for (int j = 0; j < kInFlight; ++j) {
            const uint32_t tile = base + (uint32_t)j * kCmpThreads + tid;
            const bool ticketed = tile < a.G && tile >= first_ticketed;
            const bool listed = ticketed && (!(tm[j] < thr_e) || tile == a.G - 1u);
            if (ticketed && !listed) st_relaxed_u64(a.desc + tile, desc_pack(kDescValid, 0, 0));
            const uint32_t word = __ballot_sync(kFullMask, listed);
            if (lane == 0 && (tile - lane) < a.G) bits[tile >> 5] = word;
        }
    }
    __syncthreads();                                   // the bitmap is complete (same block: visible after the barrier)
    const uint32_t nwords = (a.G + 31u) >> 5;
    uint32_t running = 0;
    for (uint32_t base = 0; base < nwords; base += kCmpThreads) {
        const uint32_t wi = base + tid;
        uint32_t word = wi < nwords ? bits[wi] : 0u;       // (written by this block before the barrier)
        const uint32_t cnt = (uint32_t)__popc(word);
        const uint32_t incl = warp_incl_scan(cnt, lane);
        if (lane == 31) s.scan_tot[warp] = incl;
        __syncthreads();
        uint32_t before = running, all = 0;
#pragma unroll
        for (int w = 0; w < kCmpWarps; ++w) {
            const uint32_t v = s.scan_tot[w];
            if (w < warp) before += v;
            all += v;
        }
        uint32_t pos = before + incl - cnt;
        if constexpr (BIG) {
            // the warp writes the tiles of its 32 words one word at a time: consecutive list entries from consecutive lanes
            for (int j = 0; j < 32; ++j) {
                const uint32_t wj = __shfl_sync(kFullMask, word, j), pj = __shfl_sync(kFullMask, pos, j);
                if ((wj >> lane) & 1u)
                    a.nelist[pj + (uint32_t)__popc(wj & ((1u << lane) - 1u))] = ((base + 32u * (uint32_t)warp + (uint32_t)j) << 5) + (uint32_t)lane;
            }
        } else {
            while (word) {
                const uint32_t bit = (uint32_t)__ffs((int)word) - 1u;
                word &= word - 1u;
                a.nelist[pos++] = (wi << 5) + bit;
            }
        }
        running += all;
        __syncthreads();
    }
    return running;
}

// Grid barrier of gradient `job` among the `expect` blocks that sum it, first half: this
// block's partial sums are written.  The last block to arrive reduces all partials on the fixed
// tree (alone: hundreds of blocks reading the same few lines at once queue up in L2), stores S,
// lists the tiles the encode pass has to read (build_tile_list), clears the count, readies the
// gradient's ticket counters and sets the gradient's flag to the launch's generation (read by
// every block when it started, bumped by the last block to leave the kernel: no state outside
// the workspace, so a launch can be replayed).  With one gradient the tiles below `tgrid` are
// encoded by the blocks that summed them last and take no ticket.
template <bool BIG>
__device__ __forceinline__ void barrier_arrive(CmpSmem& s, const CmpArgs& a, const PowTable& pw, uint32_t job, bool full, uint32_t tgrid,
                                               uint32_t expect, unsigned int gen_next, int tid, int lane, int warp) {
    Control* ctl = a.ctl;
    __syncthreads();
    if (tid == 0) {                                   // (thread 0 wrote the partials and cleared the descriptors itself)
        s.last_arrival = 0u;
        if (!s.abort_flag) {
            const unsigned int old = atom_add_acq_rel_u32(&ctl->bar_count[job], 1u);
            if (old == expect - 1u) s.last_arrival = 1u;
        }
    }
    __syncthreads();
    if (s.last_arrival) {
        float tm_ahead[kListAhead];
        tile_maxima_ahead(a, tm_ahead, tid);
        const double S = reduce_partials<BIG>(a.partials, a.G, s.s_tree, s.s_nodes, tid, lane, warp);
        __syncthreads();                                  // (the reduction's scratch becomes the list's bitmap)
        const uint32_t listed = build_tile_list<BIG>(s, a, pw, S, full ? 0u : tgrid, tm_ahead, tid, lane, warp);      // (every thread holds S)
        if (tid == 0) {
            reinterpret_cast<double*>(reinterpret_cast<unsigned char*>(ctl) + kJobSumOffset)[job] = S;
            ctl->bar_count[job] = 0u;
            ctl->tickets[job] = 0u;
            ctl->tickets1[job] = 0u;
            ctl->ne_count[job] = listed;
            st_release_u32(&ctl->bar_flag[job], gen_next);       // (the other threads' list entries were written before a block barrier)
        }
    }
}

// Second half: wait (bounded) until every block has arrived.
__device__ __forceinline__ void barrier_wait(CmpSmem& s, Control* ctl, uint32_t job, unsigned int gen_next, int tid) {
    if (tid == 0 && !s.abort_flag) {
        uint32_t spin = 0;
        while (ld_acquire_u32(&ctl->bar_flag[job]) != gen_next) {
            if (++spin > s.wait_limit) { s.abort_flag = 1u; break; }
            if (spin > 64u) __nanosleep(32);
        }
    }
    __syncthreads();
}

// After the grid barrier of gradient `job`: S (reduced by the last block to arrive) -> boundary
// table RU32(B_k) in shared memory; resets the block's per-gradient scan state.
__device__ __forceinline__ void make_table(CmpSmem& s, const CmpArgs& a, const PowTable& pw, uint32_t job, uint32_t jp,
                                           int tid, int lane, int warp) {
    const double S = __ldcg(reinterpret_cast<const double*>(reinterpret_cast<const unsigned char*>(a.ctl) + kJobSumOffset) + job);
    const bool finite = isfinite(S);
    const uint32_t skip = !finite ? 2u : (S == 0.0 ? 1u : 0u);
    if (tid <= (int)a.tau) {
        // |v| >= B_k on an fp32 |v| equals |v| >= RU32(B_k); never below the smallest denormal,
        // because an entry must also be non-zero to be kept
        const double Bk = __ddiv_rn(S, pw.P[tid]);
        s.thr[tid] = finite ? fmaxf(__double2float_ru(Bk), __int_as_float(1)) : __int_as_float(0x7f800000);
    }
    if (tid == 0) {
        // log2 S and 1 / log2 b only steer the table search (its result does not depend on them): single precision, and
        // the exponent of S taken from its bits so that sums beyond the fp32 range still give a finite estimate
        const unsigned long long sb = (unsigned long long)__double_as_longlong(S);
        const int ex = (int)((sb >> 52) & 0x7FFull) - 1023;
        const float mant = __uint_as_float(0x3F800000u | (uint32_t)((sb >> 29) & 0x7FFFFFull));      // [1, 2)
        s.thr[130] = (float)ex + __log2f(mant);
        s.thr[131] = 1.0f / __log2f((float)a.base);
        s.job_sum[jp] = S; s.job_skip[jp] = skip;
        s.ne_count = __ldcg(&a.ctl->ne_count[job]);
        s.sc_pos = 0u; s.sc_count = 0u; s.sc_words = 0u;
        s.held[0] = 0xFFFFFFFFu; s.held[1] = 0xFFFFFFFFu;
    }
    __syncthreads();
}

// Schedule of one launch.  With teams == 2 the two blocks of every SM belong to different teams;
// team t compresses gradients t, t+2, ... by itself (own barriers, tickets and prefixes), so that
// one team streams while the other sits in a control step.  A team's gradients j0 < j1 < ...:
//   sum(j0) | sum(j1), table(j0), encode(j0) | sum(j2), table(j1), place(j0), encode(j1) | ... | place(last)
// The sum pass of the next gradient runs before the encode pass of the one at hand: nobody waits at
// its grid barrier, blocks that fall behind in one pass take fewer tickets in the next, and the
// latencies of the control steps hide behind tile copies in flight.  place(j) puts the tiles of
// gradient j that were still pending at the end of its encode pass.  With a single gradient the
// block's last tile of the sum pass stays in shared memory for the encode pass.
// SEVERAL: the launch holds more than one gradient (its own instantiation: the single-gradient
// launch carries none of the team and pipelining code, and the other way round)
// BIG (one gradient only): the variant for gradients with very many tiles, where the steps that one
// block does for everybody (reducing the partials, listing the tiles, scanning the descriptors) take
// forms that cost less per tile and more to start with.
template <bool SEVERAL, bool BIG = false>
__global__ void __launch_bounds__(kCmpThreads, 2)
k_compress(const CmpBatch b, const __grid_constant__ PowTable pw) {
    extern __shared__ __align__(128) unsigned char cmp_smem_raw[];
    CmpSmem& s = *reinterpret_cast<CmpSmem*>(cmp_smem_raw);
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const uint32_t c = blockIdx.x;
#ifdef FASTSGD_TRACE
    unsigned long long* btrace = reinterpret_cast<unsigned long long*>(reinterpret_cast<unsigned char*>(b.ctl) + kJobTraceOffset) + 64u * c;
#endif

    constexpr bool full = SEVERAL;            // several gradients: every tile of every pass is handed out by ticket
    unsigned int gen_next = 0u;
    if (tid == 0) {
        gen_next = ld_acquire_u32(&b.ctl->bar_gen) + 1u;      // before this block can arrive at a barrier
        for (int st = 0; st < kSumParts; ++st) mbar_init(&s.mbar[st], 1u);
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
        s.abort_flag = 0u;
        s.wait_limit = b.wait_limit; s.try_limit = b.try_limit;
        s.held[0] = 0xFFFFFFFFu; s.held[1] = 0xFFFFFFFFu;
        uint32_t team = 0u;
        if (SEVERAL && b.teams == 2u) {       // (the host launches exactly two blocks per SM then)
            unsigned int smid;
            asm volatile("mov.u32 %0, %%smid;" : "=r"(smid));
            team = atomicAdd(b.sm_slots + (smid & 255u), 1u) & 1u;
        }
        s.team = team;
    }
    __syncthreads();
    // (one gradient: no teams, nothing of the schedule below is compiled in)
    const uint32_t team = SEVERAL ? s.team : 0u, step = SEVERAL ? b.teams : 1u;
    const uint32_t grid = SEVERAL ? gridDim.x / b.teams : gridDim.x;              // blocks of a team
    // The team's own gradients: team, team + step, ...  With two teams, to keep their control steps
    // apart and their ends together: the blocks of team 1 first take up to two tiles each of
    // gradient 0's sum pass (so team 0 runs ahead), and the team that does not own the last
    // gradient H joins H's encode pass when it is done with its own.
    const uint32_t nown = !SEVERAL ? 1u : (b.jobs > team ? (b.jobs - team + step - 1u) / step : 0u);
    const uint32_t H = SEVERAL ? b.jobs - 1u : 0u;
    const bool helper = step == 2u && (H & 1u) != team;
    const uint32_t niter = nown + (helper ? 1u : 0u);
    uint32_t parity = 0;                      // bit st: parity the next wait on stage st expects
    uint32_t pending = 0;                     // bit st: a copy into stage st has been started and not waited for
    bool aborted = false;
    // the tiles of the gradient before the one at hand that were pending at the end of its encode
    // pass: their count, that gradient's sum and status wait in shared memory
    uint32_t prev_job = 0u;
    // The pending list and the arena live across gradients: tiles [0, nprev) of the list are what
    // the previous gradient's encode pass left behind (placed after this gradient's encode pass,
    // when their prefixes have long been published), tiles [nprev, npend) belong to this gradient.
    int nprev = 0, npend = 0;
    uint32_t arena_used = 0;
    bool dense_pending = false;               // a blob of the dense path waits in the block's scratch slot
    CmpArgs a = job_view(b, 0u);

    if (step == 2u && team == 1u) {
        FSG_STAMP(8u * 7u + 0);
        const SumCursor cur = sum_begin(s, a, 0u, full, c, grid, 2u, pending, tid);
        sum_rest(s, a, 0u, full, c, grid, 2u, cur, parity, pending, tid, lane, warp);
        barrier_arrive<BIG>(s, a, pw, 0u, full, grid, gridDim.x, gen_next, tid, lane, warp);
        __syncthreads();
    }
    if (nown) {
        a = job_view(b, team);
        FSG_STAMP(8u * team + 0);
        {
            const SumCursor cur = sum_begin(s, a, team, full, c, grid, 0xFFFFFFFFu, pending, tid);
            sum_rest(s, a, team, full, c, grid, 0xFFFFFFFFu, cur, parity, pending, tid, lane, warp);
        }
        FSG_STAMP(8u * team + 1);
        barrier_arrive<BIG>(s, a, pw, team, full, grid, (step == 2u && team == 0u) ? gridDim.x : grid, gen_next, tid, lane, warp);
    }

    for (uint32_t it = 0; it < niter && !aborted; ++it) {
    const uint32_t jp = it & 1u;
    const uint32_t job = it < nown ? team + it * step : H;
    const uint32_t enc_expect = (step == 2u && job == H) ? gridDim.x : grid;      // blocks that pass through this encode pass
    a = job_view(b, job);
    __syncthreads();
    if (it + 1u < nown && !s.abort_flag) {
        // the next gradient's sum pass first: by its end the block that arrived last at this gradient's grid
        // barrier has long reduced the partial sums and listed the tiles (9 us for 1563 tiles), so that nobody waits there
        const uint32_t nj = job + step;
        const CmpArgs an = job_view(b, nj);
        FSG_STAMP(8u * nj + 0);
        const SumCursor cur = sum_begin(s, an, nj, full, c, grid, 0xFFFFFFFFu, pending, tid);
        sum_rest(s, an, nj, full, c, grid, 0xFFFFFFFFu, cur, parity, pending, tid, lane, warp);
        FSG_STAMP(8u * nj + 1);
        barrier_arrive<BIG>(s, an, pw, nj, full, grid, grid, gen_next, tid, lane, warp);
        __syncthreads();
    }
    barrier_wait(s, b.ctl, job, gen_next, tid);
    FSG_STAMP(8u * job + 3);
    if (!s.abort_flag) make_table(s, a, pw, job, jp, tid, lane, warp);
    FSG_STAMP(8u * job + 4);
    __syncthreads();
    aborted = s.abort_flag != 0u;

    if (!aborted) {
        // the block's first tile of the encode pass: with one gradient its own tile c, still there from
        // the sum pass; otherwise the first ticket it gets
        const uint32_t skip = s.job_skip[jp];
        const float thr_e = s.thr[a.tau];          // early-stop threshold tau_e
        // Tickets of the encode pass are positions in the gradient's list of tiles worth reading
        // (build_tile_list); kNoMore stands for "the list is exhausted".
        const uint32_t listed = s.ne_count;
        const bool preloaded = full;
        uint32_t g = c;
        bool have = true;
        if (full) {
            if (tid == 0) {
                const uint32_t t0 = atomicAdd(a.ticket, 1u);
                s.next_tile[1] = t0 < listed ? __ldcg(a.nelist + t0) : kNoMore;
            }
            __syncthreads();
            g = s.next_tile[1];
            have = g < a.G;
            if (have) { issue_tile(s, a, 0, g, tid); pending |= 1u; }
        }
        const CmpArgs ap = job_view(b, prev_job);
        FSG_STAMP(8u * job + 2);

        // =============================== encode pass ===============================
        // Every warp owns one slab of 1024 consecutive entries of the tile in the stage: it filters
        // it, compacts its kept entries into its own list, quantises them and forms their deltas
        // without talking to the other warps; two block barriers per tile exchange the slab
        // summaries (counts, boundary keys, largest delta -> M) and the payload bits.
        const uint32_t round_up = (1u << a.l) - 1u;
        // With one gradient the block's first tile is the one it summed last (still in shared memory);
        // every further tile is handed out by a ticket counter, so that blocks that met dense tiles
        // take fewer.  Thread 0 holds the ticket of the tile after the one at hand, taken a whole
        // iteration before it is used.
        static_assert(kStages == 1, "the encode pass keeps one tile in flight per block");
        unsigned int ticket_ahead = 0u;
        if (tid == 0 && have) ticket_ahead = atomicAdd(a.ticket, 1u);
        for (uint32_t i = 0; have && !aborted; ++i) {
            const int st = 0;
            const uint32_t par = i & 1u;
            // thread 0: which tile does the ticket taken an iteration ago stand for?  (needed before this
            // iteration's first barrier)
            uint32_t tile_ahead = kNoMore;
            if (tid == 0) tile_ahead = ticket_ahead == kNoTicket ? kNoTicket : (ticket_ahead < listed ? __ldcg(a.nelist + ticket_ahead) : kNoMore);
            if (i > 0u || preloaded) {
                if (!mbar_wait(&s.mbar[st], (parity >> st) & 1u, s.try_limit)) s.abort_flag = 1u;
                parity ^= 1u << st;
                pending &= ~(1u << st);
            }
            // ---- threshold filter on the warp's slab: kept mask, bit 4r+c <-> entry warp*1024 + r*128 + lane*4 + c
            const float* tile = s.stage[st];
            uint32_t m = 0;
            if (!skip) {
                const float4* row = reinterpret_cast<const float4*>(tile + warp * 1024) + lane;
#pragma unroll
                for (int r = 0; r < 8; ++r) {
                    const float4 q = row[r * 32];
                    if (fabsf(q.x) >= thr_e) m |= 1u << (4 * r);
                    if (fabsf(q.y) >= thr_e) m |= 2u << (4 * r);
                    if (fabsf(q.z) >= thr_e) m |= 4u << (4 * r);
                    if (fabsf(q.w) >= thr_e) m |= 8u << (4 * r);
                }
            }
            // ---- warp-local compaction in index order: per-row counts scanned over the lanes, four
            // rows per word, one byte per row; then quantisation and deltas on the warp's own list
            uint32_t ex0 = 0, ex1 = 0, tot0 = 0, tot1 = 0, slab_count = 0, slab_first = 0, slab_last = 0, slab_maxd = 0;
            if (__any_sync(kFullMask, m != 0u)) {
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
                for (int r = 0; r < 4; ++r) slab_count += ((tot0 >> (8 * r)) & 0xFFu) + ((tot1 >> (8 * r)) & 0xFFu);
                if (slab_count <= kSlabCap) {
                    uint16_t* wk = s.wkeys[warp];
                    uint32_t* wv = s.wvals[warp];
                    if (slab_count <= 128u) {
                        // up to 128 entries (measured): one round per kept entry of the lane that holds most
                        // (position = entries of earlier rows + entries of earlier lanes in the row + earlier ones of the lane in the row)
                        const uint32_t t0 = tot0 + (tot0 << 8) + (tot0 << 16) + (tot0 << 24);      // inclusive prefix of the rows' totals, a byte per row (<= 128)
                        const uint32_t t1 = tot1 + (tot1 << 8) + (tot1 << 16) + (tot1 << 24) + (t0 >> 24) * 0x01010101u;
                        const unsigned long long rowex = ((unsigned long long)(t1 - tot1 + ex1) << 32) | (t0 - tot0 + ex0);   // exclusive row prefix + lanes before
                        uint32_t mm = m;
                        while (mm) {
                            const uint32_t b = (uint32_t)__ffs((int)mm) - 1u;
                            mm &= mm - 1u;
                            const uint32_t r = b >> 2;
                            const uint32_t pos = ((uint32_t)(rowex >> (8u * r)) & 0xFFu) + (uint32_t)__popc(m & ((1u << b) - 1u) & (0xFu << (4u * r)));
                            const uint32_t k = warp * 1024 + r * 128 + lane * 4 + (b & 3u);
                            wk[pos] = (uint16_t)k;
                            wv[pos] = __float_as_uint(tile[k]);
                        }
                    } else if (m != 0u) {
                        uint32_t row_base = 0;
#pragma unroll
                        for (int r = 0; r < 8; ++r) {
                            const uint32_t tot = r < 4 ? (tot0 >> (8 * r)) & 0xFFu : (tot1 >> (8 * (r - 4))) & 0xFFu;
                            const uint32_t ex  = r < 4 ? (ex0 >> (8 * r)) & 0xFFu : (ex1 >> (8 * (r - 4))) & 0xFFu;
                            const uint32_t mr = (m >> (4 * r)) & 0xFu;
                            uint32_t pos = row_base + ex;
                            const uint32_t k0 = warp * 1024 + r * 128 + lane * 4;
                            if (mr) {
                                if (mr & 1u) { wk[pos] = (uint16_t)(k0);     wv[pos] = __float_as_uint(tile[k0]);     ++pos; }
                                if (mr & 2u) { wk[pos] = (uint16_t)(k0 + 1); wv[pos] = __float_as_uint(tile[k0 + 1]); ++pos; }
                                if (mr & 4u) { wk[pos] = (uint16_t)(k0 + 2); wv[pos] = __float_as_uint(tile[k0 + 2]); ++pos; }
                                if (mr & 8u) { wk[pos] = (uint16_t)(k0 + 3); wv[pos] = __float_as_uint(tile[k0 + 3]); ++pos; }
                            }
                            row_base += tot;
                        }
                    }
                    __syncwarp();
                    for (uint32_t j = lane; j < slab_count; j += 32) {
                        const uint32_t key = wk[j];
                        wv[j] = code_byte_of(s.thr, a.tau, __uint_as_float(wv[j]));      // value -> code byte, in place
                        if (j) slab_maxd = max(slab_maxd, key - (uint32_t)wk[j - 1]);
                    }
                    slab_maxd = __reduce_max_sync(kFullMask, slab_maxd);
                    slab_first = wk[0];
                    slab_last = wk[slab_count - 1];
                }
            }
            if (tid == 0) { s.next_tile[par] = tile_ahead; s.held[0] = g; s.held[1] = tile_ahead; }
            if (lane == 0) {
                s.sum_count[par][warp] = slab_count | (slab_count > kSlabCap ? 0x80000000u : 0u);
                s.sum_first[par][warp] = slab_first;
                s.sum_last[par][warp] = slab_last;
                s.sum_maxd[par][warp] = slab_maxd;
            }
            // barrier 1: summaries written, every thread has read its part of the stage; it also tells
            // whether the tile holds any kept entry at all
            const int any_kept = __syncthreads_or(m != 0u);
            if (s.abort_flag) { aborted = true; break; }
            // ---- every warp combines the 16 summaries (lane w <-> slab w)
            uint32_t count = 0, warp_base = 0, cnt_l = 0;
            bool overflow = false;
            if (any_kept) {
                const uint32_t sc_raw = lane < kCmpWarps ? s.sum_count[par][lane] : 0u;
                cnt_l = sc_raw & 0x7FFFFFFFu;
                count = __reduce_add_sync(kFullMask, cnt_l);
                overflow = __any_sync(kFullMask, (sc_raw >> 31) != 0u);
                const uint32_t cnt_incl = warp_incl_scan(cnt_l, lane);
                warp_base = __shfl_sync(kFullMask, cnt_incl - cnt_l, warp);      // kept entries in the slabs before mine
            }
            // The stage is free: start the copy of the next tile (reserved one iteration ago) and reserve
            // the one after -- unless the arena or the pending list will soon be full.  A block that
            // drains must not sit on a reserved tile: nobody else can publish it, so the others'
            // drains would queue up behind this one, one after the other.  Hence a block that expects
            // to drain stops reserving, finishes what it holds, drains while it holds nothing, and only
            // then takes its next ticket.
            const uint32_t worst_now = (count * (8u + a.l + (uint32_t)kGroupLog2) + 31u) >> 5;
            const uint32_t g_next = s.next_tile[par];
            const bool more = g_next < a.G;                  // (false for kNoTicket too)
            if (more) {
                if (!overflow) { issue_tile(s, a, st, g_next, tid); pending |= 1u << st; }      // (a tile too dense for the lists packs its blob in the stage first)
                if (tid == 0) {
                    const bool stop_reserving = overflow || dense_pending ||
                        npend + 3 >= kPendMax || arena_used + worst_now + 2u * kArenaReserve > kArenaWords;
                    ticket_ahead = stop_reserving ? kNoTicket : atomicAdd(a.ticket, 1u);
                }
            }

            uint32_t words = 0, M = 0, aoff = 0;
            if (count == 0u) {
                if (npend == kPendMax) { if (!drain(s, a, ap, jp, nprev, npend, tid, lane, warp)) { aborted = true; break; } nprev = 0; npend = 0; arena_used = 0; dense_pending = false; }
            } else if (!overflow) {
                const uint32_t worst = (count * (8u + a.l + (uint32_t)kGroupLog2) + 31u) >> 5;
                if (npend == kPendMax || arena_used + worst > kArenaWords) {
                    if (!drain(s, a, ap, jp, nprev, npend, tid, lane, warp)) { aborted = true; break; }
                    nprev = 0; npend = 0; arena_used = 0; dense_pending = false;
                }
                aoff = arena_used;
                uint32_t* blob = s.arena + aoff;
                // boundary deltas: a slab's first key minus the last kept key before it (0 at the tile's start),
                // found by a running maximum since the keys ascend with the slab number
                const uint32_t last_l = (lane < kCmpWarps && cnt_l) ? s.sum_last[par][lane] : 0u;
                uint32_t run = last_l;
#pragma unroll
                for (int o = 1; o < kCmpWarps; o <<= 1) {
                    const uint32_t t = __shfl_up_sync(kFullMask, run, o);
                    if (lane >= o) run = max(run, t);
                }
                const uint32_t prev_last = __shfl_up_sync(kFullMask, run, 1);
                const uint32_t bd_l = (lane < kCmpWarps && cnt_l) ? s.sum_first[par][lane] - (lane ? prev_last : 0u) : 0u;
                const uint32_t maxd_l = lane < kCmpWarps ? max(s.sum_maxd[par][lane], bd_l) : 0u;
                const uint32_t maxd = __reduce_max_sync(kFullMask, maxd_l);
                M = maxd ? (32u - __clz(maxd)) : 1u;
                const uint32_t inv_m = c_inv_m[M];
                const uint32_t my_bd = __shfl_sync(kFullMask, bd_l, warp);
                const uint32_t my_cnt = __shfl_sync(kFullMask, cnt_l, warp);
                const uint16_t* wk = s.wkeys[warp];
                const uint32_t* wv = s.wvals[warp];
                // payload bits of my slab; what the first 32 entries need again when packing stays in registers
                uint32_t d0 = 0, f0 = 0, w0 = 0;
                if ((uint32_t)lane < my_cnt) {
                    d0 = lane ? (uint32_t)wk[lane] - (uint32_t)wk[lane - 1] : my_bd;
                    f0 = flag_of(d0, a.l, inv_m);
                    w0 = ((f0 + 1u) * M + round_up) >> a.l;
                }
                const uint32_t w0_incl = warp_incl_scan(w0, lane);
                uint32_t bits = 0;
                for (uint32_t j = 32u + lane; j < my_cnt; j += 32) {
                    const uint32_t delta = (uint32_t)wk[j] - (uint32_t)wk[j - 1];
                    bits += ((flag_of(delta, a.l, inv_m) + 1u) * M + round_up) >> a.l;
                }
                if (my_cnt > 32u) bits = __reduce_add_sync(kFullMask, bits);
                bits += __shfl_sync(kFullMask, w0_incl, 31);
                if (lane == 0) s.sum_bits[par][warp] = bits;
                {
                    const uint32_t bound_words = (count * (8u + a.l + M) + 31u) >> 5;
                    for (uint32_t w = tid; w < bound_words; w += kCmpThreads) blob[w] = 0u;
                }
                __syncthreads();                   // payload bits of every slab known; blob zeroed
                const uint32_t bits_l = lane < kCmpWarps ? s.sum_bits[par][lane] : 0u;
                const uint32_t bits_incl = warp_incl_scan(bits_l, lane);
                const uint32_t bits_before = __shfl_sync(kFullMask, bits_incl - bits_l, warp);
                const uint32_t payload_bits = __shfl_sync(kFullMask, bits_incl, 31);
                const uint32_t flag_pos0 = 8u * count, delta_pos0 = flag_pos0 + a.l * count;
                words = (delta_pos0 + payload_bits + 31u) >> 5;
                // pack my slab's entries: codes | flags | deltas (most significant bit first)
                uint32_t dbase = delta_pos0 + bits_before;
                if ((uint32_t)lane < my_cnt) {
                    const uint32_t q = warp_base + lane;                  // rank of the entry in the group
                    put_byte_smem(blob, q, wv[lane] & 0xFFu);
                    put_bits_smem(blob, flag_pos0 + a.l * q, f0, a.l);
                    put_bits_smem(blob, dbase + (w0_incl - w0), d0, w0);
                }
                dbase += __shfl_sync(kFullMask, w0_incl, 31);
                for (uint32_t j0 = 32u; j0 < my_cnt; j0 += 32) {
                    const uint32_t j = j0 + lane;
                    uint32_t delta = 0, f = 0, w = 0;
                    if (j < my_cnt) {
                        delta = (uint32_t)wk[j] - (uint32_t)wk[j - 1];
                        f = flag_of(delta, a.l, inv_m);
                        w = ((f + 1u) * M + round_up) >> a.l;
                    }
                    const uint32_t w_incl = warp_incl_scan(w, lane);
                    if (j < my_cnt) {
                        const uint32_t q = warp_base + j;
                        put_byte_smem(blob, q, wv[j] & 0xFFu);
                        put_bits_smem(blob, flag_pos0 + a.l * q, f, a.l);
                        put_bits_smem(blob, dbase + (w_incl - w), delta, w);
                    }
                    dbase += __shfl_sync(kFullMask, w_incl, 31);
                }
                arena_used += words;
            } else {
                // A slab is too dense for its list: block-wide path.  The blob is packed in the stage and
                // moved to the block's slot of global scratch, where it waits like the blobs in the arena
                // (one at a time; the block takes no new ticket while it holds one, so the drain that
                // frees the slot never runs with a tile reserved).
                if (dense_pending || npend == kPendMax) {
                    if (!drain(s, a, ap, jp, nprev, npend, tid, lane, warp)) { aborted = true; break; }
                    nprev = 0; npend = 0; arena_used = 0; dense_pending = false;
                }
                aoff = kDenseMark;
                const unsigned long long wm = pack_tile_dense(&s, a.dense_scratch, a.l, a.tau, count, warp_base, m, ex0, ex1, tot0, tot1);
                words = (uint32_t)wm; M = (uint32_t)(wm >> 32);
                {
                    uint32_t* slot_blob = reinterpret_cast<uint32_t*>(a.dense_scratch + (uint64_t)blockIdx.x * kDenseScratchBytes);
                    const uint32_t* stage_blob = reinterpret_cast<const uint32_t*>(s.stage[0]);
                    for (uint32_t i2 = tid; i2 < words; i2 += kCmpThreads) slot_blob[i2] = stage_blob[i2];
                }
                dense_pending = true;
                __syncthreads();                     // the stage is free
                if (more) {                          // (generic-proxy writes before an async-proxy one)
                    if (tid == 0) asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
                    issue_tile(s, a, st, g_next, tid); pending |= 1u << st;
                }
            }
            if (tid == 0) {
                st_relaxed_u64(a.desc + g, desc_pack(kDescValid, count, words));
                s.pend_g[npend] = g;
                s.pend_cm[npend] = count ? (count | (M << 24)) : 0u;
                s.pend_words[npend] = words;
                s.pend_off[npend] = aoff;
            }
            ++npend;
            if (g_next == kNoTicket) {
                // Nothing reserved: drain now.  Once the waiting half is over nobody can be held up by
                // this block any more, so it takes its next ticket and starts that copy before it places its blobs.
                __syncthreads();
                if (npend > 0 && !drain_wait(s, a, ap, nprev, npend, tid, lane, warp)) { aborted = true; break; }
                if (tid == 0) {
                    const uint32_t t1 = atomicAdd(a.ticket, 1u);
                    s.next_tile[par] = t1 < listed ? __ldcg(a.nelist + t1) : kNoMore;
                }
                __syncthreads();
                g = s.next_tile[par];
                have = g < a.G;
                if (have) {
                    issue_tile(s, a, st, g, tid); pending |= 1u << st;
                    if (tid == 0) ticket_ahead = atomicAdd(a.ticket, 1u);
                }
                if (npend > 0) drain_place(s, a, ap, jp, nprev, npend, tid, lane, warp);
                nprev = 0; npend = 0; arena_used = 0; dense_pending = false;
                __syncthreads();                   // next_tile[par] is rewritten two iterations from now at the earliest
            } else {
                g = g_next;
                have = more;
            }
        }
        FSG_STAMP(8u * job + 5);
        // this block's tiles of the gradient are published: count it; the last block through computes
        // the prefixes for everybody
        if (tid == 0) {
            s.publisher = 0u;
            if (!aborted) {
                const unsigned int old = atom_add_acq_rel_u32(a.enc_done, 1u);      // this block's descriptors before its count
                if (old == enc_expect - 1u) *a.enc_done = 0u;
                // the launch's last gradient: the first block through follows the others; else the last one scans
                if constexpr (BIG) s.publisher = old < min(kScanParts, enc_expect) ? old + 1u : 0u;      // (one gradient: the first blocks through share the scan)
                else s.publisher = (job == H ? old == 0u : old == enc_expect - 1u) ? 1u : 0u;
            }
        }
        __syncthreads();
        if (s.publisher) {
            if constexpr (BIG) {
                // (the per-SM counters of the two-team launches are not in use here: their place holds the segment totals)
                publish_part(s, a, reinterpret_cast<unsigned long long*>(b.sm_slots), s.publisher - 1u, min(kScanParts, enc_expect), tid, lane, warp);
            } else {
                // (following the others; it starts when the tickets run out, with most descriptors published: large steps when
                // a single gradient has thousands of them, else small ones, so that what is complete is published at once;
                // measured: 2^26 entries -3 %, 50 M and the four-gradient launch +1 % with large steps)
                if (job == H) {
                    if (!SEVERAL && a.G >= 8u * kCmpThreads) publish_prefixes<true, kDrainChunks>(s, a, tid, lane, warp);
                    else publish_prefixes<true, 1>(s, a, tid, lane, warp);
                }
                else publish_prefixes<false, kDrainChunks>(s, a, tid, lane, warp);
            }
            FSG_STAMP(7);
        }
        // place what the previous gradient left behind; what this one leaves waits for the next turn
        if (!aborted && nprev > 0) {
            if (!drain_final(s, ap, jp ^ 1u, nprev, tid, lane, warp)) { aborted = true; break; }
            const int rest = npend - nprev;
            uint32_t e_g = 0, e_cm = 0, e_w = 0, e_o = 0;
            if (tid < rest) { e_g = s.pend_g[nprev + tid]; e_cm = s.pend_cm[nprev + tid]; e_w = s.pend_words[nprev + tid]; e_o = s.pend_off[nprev + tid]; }
            __syncthreads();
            if (tid < rest) { s.pend_g[tid] = e_g; s.pend_cm[tid] = e_cm; s.pend_words[tid] = e_w; s.pend_off[tid] = e_o; }
            __syncthreads();
            npend = rest;
            dense_pending = false;
            for (int p = 0; p < npend; ++p) dense_pending = dense_pending || s.pend_off[p] == kDenseMark;
        }
        nprev = npend;
        if (npend == 0) arena_used = 0;
        prev_job = job;
    }
    }   // jobs

    if (!aborted && nprev > 0) {
        __syncthreads();                           // pending list written by thread 0
        if (!drain_final(s, job_view(b, prev_job), (niter - 1u) & 1u, nprev, tid, lane, warp)) aborted = true;
    }
    FSG_STAMP(6);   // (slot 6 of the first gradient: end of the launch's last drain)

    if (aborted) {
        // give up: record it, unblock the others, wait for this block's copies, mark every stream of
        // the launch as timed out, return.
        __syncthreads();
        if (tid == 0) {
            atomicExch(&a.ctl->error, (unsigned)kStTimeout);
            // (in the sum pass nobody waits for descriptors yet)
            if (s.held[0] < a.G) st_relaxed_u64(a.desc + s.held[0], desc_pack(kDescPoison, 0, 0));
            if (s.held[1] < a.G) st_relaxed_u64(a.desc + s.held[1], desc_pack(kDescPoison, 0, 0));
            for (int st = 0; st < kSumParts; ++st)
                if (pending & (1u << st)) mbar_wait(&s.mbar[st], (parity >> st) & 1u, s.try_limit);
            write_timeout_headers(b);
        }
        __syncthreads();
    }

    // the last block to leave readies the workspace for the next launch
    if (tid == 0) {
        const unsigned int old = atom_add_acq_rel_u32(&b.ctl->exit_count, 1u);
        if (old == gridDim.x - 1u) {
            // a block that did not give up may have written an OK header after the others marked the streams: the
            // last block out (it sees every other block's writes) has the final word
            if (ld_acquire_u32(&b.ctl->error) != 0u) write_timeout_headers(b);
            b.ctl->exit_count = 0u;
            if (b.teams == 2u) for (int i = 0; i < 256; ++i) b.sm_slots[i] = 0u;
            if constexpr (BIG) for (int i = 0; i < 2 * (int)kScanParts; ++i) b.sm_slots[i] = 0u;
            st_release_u32(&b.ctl->bar_gen, gen_next);
        }
    }
}

}  // namespace fsg
