// Shared definitions of the CUDA side: stream constants, the workspace layout and small
// device helpers.  sm_100a only.
#pragma once

#include <cuda_runtime.h>
#include <stdint.h>

namespace fsg {

constexpr uint32_t kMagic       = 0x31475346u;   // "FSG1"
constexpr uint32_t kVersion     = 1u;
constexpr uint32_t kHeaderBytes = 64u;
constexpr int      kMaxTau      = 128;

// The sum tree is cut into aligned chunks of 2^14 entries: one fp64 partial per chunk.
constexpr int      kChunkLog2   = 14;
constexpr uint32_t kChunk       = 1u << kChunkLog2;

constexpr int kStOk = 0, kStNonfinite = 1, kStCapacity = 2, kStTimeout = 3;
constexpr int kStBadMagic = 16, kStBadVersion = 17, kStBadStatus = 18, kStNMismatch = 19,
              kStParamMismatch = 20, kStTruncated = 21, kStBadDirectory = 22, kStBadKey = 23,
              kStBadCode = 24;

// b^k, k = 0..tau, by the recurrence P_k = P_{k-1} * b in fp64 (a function of the
// parameters alone; passed to the kernels by value).
struct PowTable {
    double P[kMaxTau + 1];
};

// Control block at the start of the workspace.
struct Control {
    unsigned int       done;           // blocks of the sum kernel that have finished (self-resetting)
    unsigned int       ticket;         // (unused)
    unsigned int       error;          // encode: non-zero once a bounded wait ran out
    unsigned int       skip;           // (unused)
    unsigned long long decode_status;  // min over failures of (group << 32 | key index << 8 | status)
    double             sum;            // S
    unsigned int       bar_gen;        // launches of k_compress that have finished
    unsigned int       exit_count;     // blocks of the running k_compress launch that have finished (self-resetting)
    unsigned int       dq[6];          // decoder work queue: pushed, taken, done, exited, reserved (zero between launches)
    unsigned int       tickets[8];     // encode pass: next tile of each gradient of the launch
    unsigned int       tickets1[8];    // sum pass: the same (zero between launches)
    unsigned int       enc_done[8];    // encode pass: blocks that have published all their tiles of each gradient (self-resetting)
    unsigned int       bar_count[8];   // blocks that have finished each gradient's sum pass (self-resetting)
    unsigned int       bar_flag[8];    // set to bar_gen + 1 by the last of them: that gradient's partial sums are complete
    unsigned int       ne_count[8];    // tiles of each gradient the encode pass has to read (written before bar_flag)
};
static_assert(sizeof(Control) == 256, "control block is 256 bytes");

constexpr uint64_t kThrOffset      = 256;    // float thr[132]: RU32(B_k)
constexpr uint64_t kJobSumOffset   = 800;    // double S[8]: the sum of each gradient of a k_compress launch
constexpr uint64_t kTraceOffset    = 1024;   // u64 trace[<=496][8]: per-block %globaltimer stamps (profiling aid)
constexpr uint64_t kQueueOffset    = 32768;  // u32 queue[2^17]: decoder's grid-wide queue of groups (zero between launches)
constexpr uint64_t kQueueBytes     = 4ull << 17;
constexpr uint64_t kJobTraceOffset = kQueueOffset + kQueueBytes;  // u64 [320 blocks][8 gradients][8]: k_compress stamps (profiling aid)
constexpr uint64_t kJobTraceBytes  = 320ull * 8ull * 8ull * 8ull;
constexpr uint64_t kSmSlotOffset   = kJobTraceOffset + kJobTraceBytes;  // u32 [256]: blocks of the running launch seen on each SM (zero between launches)
constexpr uint64_t kSmSlotBytes    = 1024;
constexpr uint64_t kKvPartialsOffset = kSmSlotOffset + kSmSlotBytes;   // double [2^17]: chunk nodes of the key-value encoder's sum (zero between launches)
constexpr uint64_t kKvPartialsBytes  = 8ull << 17;
constexpr uint64_t kKvAggOffset    = kKvPartialsOffset + kKvPartialsBytes;   // u64 [512]: per-block totals of the key-value encoder
constexpr uint64_t kKvAggBytes     = 8ull * 512ull;
constexpr uint64_t kPartialsOffset = kKvAggOffset + kKvAggBytes;  // per gradient of a launch: double partial[chunks]; then u64 desc[G]; then u64 prefix[G]; then float tmax[G]; then u32 nelist[G]; then u32 nebits[ceil(G / 32)]

struct WorkspaceView {
    Control*            ctl;
    float*              thr;
    double*             partials;
    unsigned long long* desc;
    unsigned long long* prefix;
    float*              tmax;
    uint32_t*           nelist;
    uint32_t*           nebits;
};

__host__ __device__ inline uint64_t ceil_div_u64(uint64_t a, uint64_t b) { return (a + b - 1) / b; }

// ---- look-back descriptors: status(2) | count(31) | words(31) -----------------------------
constexpr unsigned long long kDescInvalid = 0ull, kDescAggregate = 1ull, kDescPrefix = 2ull, kDescPoison = 3ull;
constexpr unsigned long long kDescValueMask = (1ull << 62) - 1ull;

__device__ __forceinline__ unsigned long long desc_pack(unsigned long long st, uint32_t count, uint32_t words) {
    return (st << 62) | ((unsigned long long)count << 31) | (unsigned long long)words;
}
__device__ __forceinline__ uint32_t desc_count(unsigned long long v) { return (uint32_t)((v >> 31) & 0x7FFFFFFFull); }
__device__ __forceinline__ uint32_t desc_words(unsigned long long v) { return (uint32_t)(v & 0x7FFFFFFFull); }

__device__ __forceinline__ unsigned long long ld_acquire_u64(const unsigned long long* p) {
    unsigned long long v;
    asm volatile("ld.acquire.gpu.global.u64 %0, [%1];" : "=l"(v) : "l"(p) : "memory");
    return v;
}
__device__ __forceinline__ void st_release_u64(unsigned long long* p, unsigned long long v) {
    asm volatile("st.release.gpu.global.u64 [%0], %1;" ::"l"(p), "l"(v) : "memory");
}

__device__ __forceinline__ uint32_t bswap32(uint32_t x) { return __byte_perm(x, 0, 0x0123); }

// bits [pos, pos+nb) of a most-significant-bit-first sequence stored as bytes; `words` is the
// sequence viewed as little-endian 32-bit words, `nwords` its length.  nb <= 32.
__device__ __forceinline__ uint32_t get_bits_be(const uint32_t* __restrict__ words, uint32_t nwords,
                                                uint32_t pos, uint32_t nb) {
    uint32_t wi = pos >> 5, sh = pos & 31u;
    uint32_t w0 = wi < nwords ? bswap32(__ldg(words + wi)) : 0u;
    uint32_t w1 = (wi + 1u) < nwords ? bswap32(__ldg(words + wi + 1u)) : 0u;
    unsigned long long both = ((unsigned long long)w0 << 32) | w1;
    if (nb == 0) return 0u;
    return (uint32_t)((both >> (64u - sh - nb)) & ((nb >= 32u) ? 0xFFFFFFFFull : ((1ull << nb) - 1ull)));
}

}  // namespace fsg
