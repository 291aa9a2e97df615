// Small device helpers shared by the encoder and the decoder: group size, bit packing into
// shared memory, warp scan.  sm_100a only.
#pragma once

#include "common.cuh"
#include "sum.cuh"

namespace fsg {

constexpr int      kGroupLog2    = 14;            // the group size the kernels are built for: T = 2^14 indices
constexpr uint32_t kGroup        = 1u << kGroupLog2;

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

}  // namespace fsg
