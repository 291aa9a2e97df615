// Small device helpers shared by the encoder and the decoder: group size, bit packing into
// shared memory, warp scan.  sm_100a only.
#pragma once

#include "common.cuh"
#include "sum.cuh"

namespace fsg {

constexpr int      kGroupLog2    = 14;            // the group size the kernels are built for: T = 2^14 indices
constexpr uint32_t kGroup        = 1u << kGroupLog2;

// OR `nb` bits (value < 2^nb, nb <= 32) into a zeroed most-significant-bit-first sequence held
// as big-endian-valued 32-bit words in shared memory.  Branch-free up to the second word: the
// field is placed in a 64-bit window that starts at its first word.
__device__ __forceinline__ void put_bits_smem(uint32_t* blob, uint32_t pos, uint32_t value, uint32_t nb) {
    if (nb == 0) return;
    const uint32_t wi = pos >> 5, sh = pos & 31u;
    const unsigned long long win = (unsigned long long)value << (64u - sh - nb);
    atomicOr(&blob[wi], (uint32_t)(win >> 32));
    const uint32_t lo = (uint32_t)win;
    if (lo) atomicOr(&blob[wi + 1], lo);
}

// the same for a byte at a byte position (never crosses a word)
__device__ __forceinline__ void put_byte_smem(uint32_t* blob, uint32_t byte_index, uint32_t value) {
    atomicOr(&blob[byte_index >> 2], value << (24u - 8u * (byte_index & 3u)));
}

__device__ __forceinline__ uint32_t warp_incl_scan(uint32_t v, int lane) {
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) {
        uint32_t t = __shfl_up_sync(kFullMask, v, o);
        if (lane >= o) v += t;
    }
    return v;
}

}  // namespace fsg
