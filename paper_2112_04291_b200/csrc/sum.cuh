// Step 1 of Algorithm 1: sum = sum_i |v_i|, and the boundary table that follows from it.
//
// The sum is defined on the balanced binary tree over index ranges aligned to powers of two
// (leaf = |v_i| widened to fp64, zero beyond n), every node one IEEE fp64 addition.  Any tiling
// by aligned power-of-two ranges reproduces that tree exactly, so the result does not depend
// on the grid: a thread reduces 4 consecutive entries, a warp 8 rows of 128 entries (1024),
// a block of 16 warps one chunk of 2^14, and the last block to finish reduces the per-chunk
// partials in the same tree order and derives B_k = sum / b^k.
#pragma once

#include "common.cuh"

namespace fsg {

constexpr int kSumThreads = 512;
constexpr unsigned kFullMask = 0xFFFFFFFFu;

__device__ __forceinline__ double abs_sum4(float4 v) {
    double a = (double)fabsf(v.x), b = (double)fabsf(v.y), c = (double)fabsf(v.z), d = (double)fabsf(v.w);
    return __dadd_rn(__dadd_rn(a, b), __dadd_rn(c, d));
}

// float4 at element index e (multiple of 4) of a 16-byte aligned array of n floats, zero beyond n
__device__ __forceinline__ float4 load4_guarded(const float* __restrict__ g, uint64_t e, uint64_t n) {
    if (e + 4 <= n) return __ldg(reinterpret_cast<const float4*>(g + e));
    float4 v = make_float4(0.f, 0.f, 0.f, 0.f);
    if (e < n) v.x = __ldg(g + e);
    if (e + 1 < n) v.y = __ldg(g + e + 1);
    if (e + 2 < n) v.z = __ldg(g + e + 2);
    return v;
}

// x[r] = tree node of this lane's 4 entries in row r (128 entries per row, 8 consecutive rows).
// Returns, in every lane, the tree node of the whole 1024-entry slab.
__device__ __forceinline__ double warp_slab_tree(const double (&x)[8], int lane) {
    const bool b0 = lane & 1, b1 = lane & 2, b2 = lane & 4;
    double y[4], z[2], u;
#pragma unroll
    for (int i = 0; i < 4; ++i) {   // lanes 2k,2k+1: 8 entries of row i (even lane) / i+4 (odd lane)
        double keep = b0 ? x[i + 4] : x[i], send = b0 ? x[i] : x[i + 4];
        y[i] = __dadd_rn(keep, __shfl_xor_sync(kFullMask, send, 1));
    }
#pragma unroll
    for (int i = 0; i < 2; ++i) {   // 16 entries of row i + 2*b1 + 4*b0
        double keep = b1 ? y[i + 2] : y[i], send = b1 ? y[i] : y[i + 2];
        z[i] = __dadd_rn(keep, __shfl_xor_sync(kFullMask, send, 2));
    }
    {                               // 32 entries of row b2 + 2*b1 + 4*b0
        double keep = b2 ? z[1] : z[0], send = b2 ? z[0] : z[1];
        u = __dadd_rn(keep, __shfl_xor_sync(kFullMask, send, 4));
    }
    u = __dadd_rn(u, __shfl_xor_sync(kFullMask, u, 8));    // 64 entries
    u = __dadd_rn(u, __shfl_xor_sync(kFullMask, u, 16));   // the row (128)
    u = __dadd_rn(u, __shfl_xor_sync(kFullMask, u, 4));    // rows 2k, 2k+1
    u = __dadd_rn(u, __shfl_xor_sync(kFullMask, u, 2));    // 4 rows
    u = __dadd_rn(u, __shfl_xor_sync(kFullMask, u, 1));    // 8 rows = 1024 entries
    return u;
}

// The same for half a slab: x[r] = tree node of this lane's 4 entries in row r of 4 consecutive rows.
// Returns, in every lane, the tree node of the 512 entries.
__device__ __forceinline__ double warp_halfslab_tree(const double (&x)[4], int lane) {
    const bool b0 = lane & 1, b1 = lane & 2;
    double y[2], z, u;
#pragma unroll
    for (int i = 0; i < 2; ++i) {   // lanes 2k,2k+1: 8 entries of row i (even lane) / i+2 (odd lane)
        double keep = b0 ? x[i + 2] : x[i], send = b0 ? x[i] : x[i + 2];
        y[i] = __dadd_rn(keep, __shfl_xor_sync(kFullMask, send, 1));
    }
    {                               // 16 entries of row b1 + 2*b0
        double keep = b1 ? y[1] : y[0], send = b1 ? y[0] : y[1];
        z = __dadd_rn(keep, __shfl_xor_sync(kFullMask, send, 2));
    }
    u = __dadd_rn(z, __shfl_xor_sync(kFullMask, z, 4));    // 32 entries
    u = __dadd_rn(u, __shfl_xor_sync(kFullMask, u, 8));    // 64 entries
    u = __dadd_rn(u, __shfl_xor_sync(kFullMask, u, 16));   // the row (128)
    u = __dadd_rn(u, __shfl_xor_sync(kFullMask, u, 2));    // rows 2k, 2k+1
    u = __dadd_rn(u, __shfl_xor_sync(kFullMask, u, 1));    // 4 rows = 512 entries
    return u;
}

// x[j] = the value at position 32 j + lane of 512 consecutive positions (16 rows of 32).  Returns,
// in every lane, the tree node of the 512 positions (rows first, then the rows pairwise).
__device__ __forceinline__ double warp_rows16_tree(const double (&x)[16], int lane) {
    const bool b0 = lane & 1, b1 = lane & 2, b2 = lane & 4, b3 = lane & 8;
    double y[8], z[4], w[2], u;
#pragma unroll
    for (int i = 0; i < 8; ++i) {   // lanes 2k,2k+1: positions 2k,2k+1 of row i (even lane) / i+8 (odd lane)
        double keep = b0 ? x[i + 8] : x[i], send = b0 ? x[i] : x[i + 8];
        y[i] = __dadd_rn(keep, __shfl_xor_sync(kFullMask, send, 1));
    }
#pragma unroll
    for (int i = 0; i < 4; ++i) {   // 4 positions of row i + 4*b1 + 8*b0
        double keep = b1 ? y[i + 4] : y[i], send = b1 ? y[i] : y[i + 4];
        z[i] = __dadd_rn(keep, __shfl_xor_sync(kFullMask, send, 2));
    }
#pragma unroll
    for (int i = 0; i < 2; ++i) {   // 8 positions of row i + 2*b2 + 4*b1 + 8*b0
        double keep = b2 ? z[i + 2] : z[i], send = b2 ? z[i] : z[i + 2];
        w[i] = __dadd_rn(keep, __shfl_xor_sync(kFullMask, send, 4));
    }
    {                               // 16 positions of row b3 + 2*b2 + 4*b1 + 8*b0
        double keep = b3 ? w[1] : w[0], send = b3 ? w[0] : w[1];
        u = __dadd_rn(keep, __shfl_xor_sync(kFullMask, send, 8));
    }
    u = __dadd_rn(u, __shfl_xor_sync(kFullMask, u, 16));   // the row
    u = __dadd_rn(u, __shfl_xor_sync(kFullMask, u, 8));    // rows 2k, 2k+1
    u = __dadd_rn(u, __shfl_xor_sync(kFullMask, u, 4));    // 4 rows
    u = __dadd_rn(u, __shfl_xor_sync(kFullMask, u, 2));    // 8 rows
    u = __dadd_rn(u, __shfl_xor_sync(kFullMask, u, 1));    // 16 rows = 512 positions
    return u;
}

// tree over the 32 lanes' values (lane = position)
__device__ __forceinline__ double warp_tree(double u, int width = 32) {
    for (int o = 1; o < width; o <<= 1) u = __dadd_rn(u, __shfl_xor_sync(kFullMask, u, o));
    return u;
}

struct SumArgs {
    const float*        grad;
    uint64_t            n;
    uint32_t            chunks;      // ceil(n / 2^14)
    uint32_t            groups;      // look-back descriptors to clear (0: none)
    uint32_t            tau;
    Control*            ctl;
    float*              thr;
    double*             partials;
    unsigned long long* desc;
    double*             sum_out;     // optional copy of the sum
};

__global__ void __launch_bounds__(kSumThreads)
k_abs_sum(const SumArgs a, const __grid_constant__ PowTable pw) {
    __shared__ double s_warp[2][kSumThreads / 32];
    __shared__ double s_tree[kSumThreads / 32];
    __shared__ bool s_last;
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;

    // the look-back state of the encode kernel that follows on the same stream
    for (uint32_t i = blockIdx.x * kSumThreads + tid; i < a.groups; i += gridDim.x * kSumThreads) a.desc[i] = 0ull;

    // chunks are visited from the end of the array towards its start, so that the entries the
    // encode kernel reads first are the ones most recently brought into L2
    int it = 0;
    for (uint32_t c = blockIdx.x; c < a.chunks; c += gridDim.x, ++it) {
        const uint32_t chunk = a.chunks - 1u - c;
        const uint64_t base = ((uint64_t)chunk << kChunkLog2) + (uint64_t)warp * 1024u + (uint64_t)lane * 4u;
        double x[8];
        if ((((uint64_t)chunk + 1u) << kChunkLog2) <= a.n) {
            float4 v[8];
#pragma unroll
            for (int r = 0; r < 8; ++r) v[r] = __ldg(reinterpret_cast<const float4*>(a.grad + base + r * 128));
#pragma unroll
            for (int r = 0; r < 8; ++r) x[r] = abs_sum4(v[r]);
        } else {
#pragma unroll
            for (int r = 0; r < 8; ++r) x[r] = abs_sum4(load4_guarded(a.grad, base + r * 128, a.n));
        }
        double u = warp_slab_tree(x, lane);
        if (lane == 0) s_warp[it & 1][warp] = u;
        __syncthreads();
        if (warp == 0) {
            double t = lane < kSumThreads / 32 ? s_warp[it & 1][lane] : 0.0;
            t = warp_tree(t, kSumThreads / 32);
            if (lane == 0) a.partials[chunk] = t;
        }
    }

    // last block to finish reduces the partials
    __threadfence();
    __syncthreads();
    if (tid == 0) {
        unsigned int prev = atomicAdd(&a.ctl->done, 1u);
        s_last = (prev == gridDim.x - 1);
    }
    __syncthreads();
    if (!s_last) return;
    __threadfence();

    // per-thread aligned run of `run` partials (a power of two), then the tree over threads
    uint32_t n2 = 1;
    while (n2 < a.chunks) n2 <<= 1;
    const uint32_t run = n2 > (uint32_t)kSumThreads ? n2 / kSumThreads : 1u;
    double acc = 0.0;
    {
        // pairwise summation of a run with a binary counter: level[b] holds the pending node of
        // 2^b partials; a new leaf merges upwards while the matching bit of its index is set
        double level[20];
        const uint64_t lo = (uint64_t)tid * run;
        for (uint32_t i0 = 0; i0 < run; i0 += 8) {
            double leaf[8];          // eight independent L2 loads in flight
#pragma unroll
            for (int k = 0; k < 8; ++k) {
                const uint64_t idx = lo + i0 + k;
                leaf[k] = (i0 + k < run && idx < a.chunks) ? __ldcg(a.partials + idx) : 0.0;
            }
#pragma unroll
            for (int k = 0; k < 8; ++k) {
                const uint32_t i = i0 + k;
                if (i < run) {
                    double node = leaf[k];
#pragma unroll
                    for (int b = 0; b < 20; ++b) {
                        if ((i >> b) & 1u) node = __dadd_rn(level[b], node);
                        else { level[b] = node; break; }
                    }
                    acc = node;   // after the last leaf (i = run-1, all low bits set) this is the run's node
                }
            }
        }
    }
    acc = warp_tree(acc);
    if (lane == 0) s_tree[warp] = acc;
    __syncthreads();
    if (warp == 0) {
        double t = lane < kSumThreads / 32 ? s_tree[lane] : 0.0;
        t = warp_tree(t, kSumThreads / 32);
        if (lane == 0) s_tree[0] = t;
    }
    __syncthreads();
    const double S = s_tree[0];
    const bool finite = isfinite(S);
    if (tid <= (int)a.tau) {
        // B_k = S / b^k; the compare |v| >= B_k on an fp32 |v| equals |v| >= RU32(B_k)
        // (never below the smallest denormal: an entry must also be non-zero to be kept)
        double Bk = __ddiv_rn(S, pw.P[tid]);
        a.thr[tid] = finite ? fmaxf(__double2float_ru(Bk), __int_as_float(1)) : __int_as_float(0x7f800000);
    }
    if (tid == 0) {
        a.ctl->sum = S;
        a.ctl->skip = !finite ? 2u : (S == 0.0 ? 1u : 0u);
        a.ctl->ticket = 0u;
        a.ctl->error = 0u;
        a.ctl->done = 0u;
        if (a.sum_out) *a.sum_out = S;
    }
}

}  // namespace fsg
