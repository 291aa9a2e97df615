// C-ABI shim: argument checks, workspace bookkeeping and kernel launches on the caller's
// stream.  No computation of the path happens here except the parameter-only table b^k.
#include "../../include/fastsgd.h"
#include "../../include/fastsgd_debug.h"

#include <atomic>
#include <cmath>
#include <cstring>
#include <mutex>
#include <vector>

#include "common.cuh"
#include "sum.cuh"
#include "bits.cuh"
#include "compress.cuh"
#include "keys_paper.cuh"
#include "kv.cuh"
#include "decode.cuh"

namespace {

using namespace fsg;

// Per device: the registered workspace and what the launches need to know about the GPU.
struct State {
    void*      ws = nullptr;
    uint64_t   ws_bytes = 0;
    int        sm_count = 0;
    int        sum_blocks_per_sm = 0;
    int        dec_blocks_per_sm = 0;
    int        cmp_blocks_per_sm = 0;
    int        kv_blocks_per_sm = 0;
    bool       attrs_set = false;
    bool       timed_out = false;          // a status query saw FASTSGD_ST_TIMEOUT: the workspace's counters are not at rest
};
// Process-wide test settings (fastsgd_debug_*).
struct Tunables {
    uint32_t   grid_override = 0;          // blocks of the encoders' launches (0: as many as are resident); tests only
    uint32_t   wait_limit = kWaitLimit;    // bounded waits of the kernels (shortened only by fastsgd_debug_set_wait_limits)
    uint32_t   try_limit = kTryLimit;
    uint32_t   dec_spin_limit = kDecSpinLimit;
};
constexpr int kMaxDevices = 64;
std::mutex g_mu;                           // guards everything below (host side only: the calls of one device share its workspace)
State      g_states[kMaxDevices];
Tunables   g_tun;

// the state of the current device (caller holds g_mu)
State* device_state() {
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess) { cudaGetLastError(); dev = 0; }      // (no device at all: the argument checks still answer)
    if (dev < 0 || dev >= kMaxDevices) return nullptr;
    return &g_states[dev];
}
#define FSG_DEVICE_STATE() State* sp_ = device_state(); if (!sp_) return FASTSGD_E_CUDA; State& g_state = *sp_

std::atomic<uint64_t> g_launches{0};

// optional per-kernel timing (profiling aid)
struct TimedLaunch { int kernel; cudaEvent_t start, stop; };
bool g_timing = false;
std::vector<TimedLaunch> g_timed;
std::vector<std::pair<cudaEvent_t, cudaEvent_t>> g_event_pool;

struct LaunchTimer {
    bool active = false; TimedLaunch t{}; cudaStream_t st;
    LaunchTimer(int kernel, cudaStream_t s) : st(s) {
        if (!g_timing) return;
        if (g_event_pool.empty()) {
            if (cudaEventCreate(&t.start) != cudaSuccess || cudaEventCreate(&t.stop) != cudaSuccess) return;
        } else { t.start = g_event_pool.back().first; t.stop = g_event_pool.back().second; g_event_pool.pop_back(); }
        t.kernel = kernel; active = true;
        cudaEventRecord(t.start, st);
    }
    ~LaunchTimer() { if (active) { cudaEventRecord(t.stop, st); g_timed.push_back(t); } }
};

int check_params(const fastsgd_params* p, PowTable* pw) {
    if (!p) return FASTSGD_E_NULL;
    if (!(p->base > 1.0) || !std::isfinite(p->base)) return FASTSGD_E_BAD_PARAM;
    if (p->tau < 1 || p->tau > (uint32_t)kMaxTau) return FASTSGD_E_BAD_PARAM;
    if (p->flag_bits < 1 || p->flag_bits > 5) return FASTSGD_E_BAD_PARAM;
    if (p->group_log2 < 1 || p->group_log2 > 20) return FASTSGD_E_BAD_PARAM;
    if (p->reserved != 0) return FASTSGD_E_BAD_PARAM;
    PowTable local;
    PowTable& t = pw ? *pw : local;
    volatile double acc = 1.0;            // one rounded fp64 product per step
    t.P[0] = 1.0;
    for (uint32_t k = 1; k <= (uint32_t)kMaxTau; ++k) {
        if (k <= p->tau) { acc = acc * p->base; t.P[k] = acc; }
        else t.P[k] = t.P[p->tau];
    }
    if (!std::isfinite(t.P[p->tau])) return FASTSGD_E_BAD_PARAM;
    return FASTSGD_OK;
}

int check_n(uint64_t n) { return (n == 0 || n >= (1ull << 31)) ? FASTSGD_E_BAD_N : FASTSGD_OK; }

uint64_t groups_of(uint64_t n, uint32_t group_log2) { return (n + (1ull << group_log2) - 1) >> group_log2; }
uint64_t chunks_of(uint64_t n) { return (n + kChunk - 1) >> kChunkLog2; }

uint64_t bound_bytes(uint64_t n, const fastsgd_params* p) {
    const uint64_t T = 1ull << p->group_log2, G = groups_of(n, p->group_log2);
    const uint64_t per_group_words = (T * (8ull + p->flag_bits + p->group_log2) + 31ull) / 32ull;
    return kHeaderBytes + 8ull * G + 4ull * G * per_group_words;
}

uint64_t ws_dense_offset(uint64_t n, uint32_t group_log2) {
    // partials, descriptors, prefixes, tile maxima, the list of tiles to encode and its bitmap for every gradient one launch can take
    const uint64_t G = groups_of(n, group_log2);
    const uint64_t b = kPartialsOffset + (uint64_t)kCmpMaxJobs * (8ull * chunks_of(n) + 24ull * G + 4ull * ((G + 31ull) >> 5));
    return (b + 255ull) & ~255ull;
}

uint64_t ws_bytes_for(uint64_t n, uint32_t group_log2) {
    return ws_dense_offset(n, group_log2) + (uint64_t)kMaxCtas * kDenseScratchBytes;
}

WorkspaceView view(void* ws, uint64_t n, uint32_t group_log2 = kGroupLog2) {
    WorkspaceView v;
    unsigned char* base = static_cast<unsigned char*>(ws);
    v.ctl = reinterpret_cast<Control*>(base);
    v.thr = reinterpret_cast<float*>(base + kThrOffset);
    v.partials = reinterpret_cast<double*>(base + kPartialsOffset);
    v.desc = reinterpret_cast<unsigned long long*>(base + kPartialsOffset + (uint64_t)kCmpMaxJobs * 8ull * chunks_of(n));
    v.prefix = v.desc + (uint64_t)kCmpMaxJobs * groups_of(n, group_log2);
    v.tmax = reinterpret_cast<float*>(v.prefix + (uint64_t)kCmpMaxJobs * groups_of(n, group_log2));
    v.nelist = reinterpret_cast<uint32_t*>(v.tmax + (uint64_t)kCmpMaxJobs * groups_of(n, group_log2));
    v.nebits = v.nelist + (uint64_t)kCmpMaxJobs * groups_of(n, group_log2);
    return v;
}

int ensure_device_setup() {
    // caller holds g_mu; once per device
    FSG_DEVICE_STATE();
    if (g_state.attrs_set) return FASTSGD_OK;
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess) return FASTSGD_E_CUDA;
    int sms = 0;
    if (cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess) return FASTSGD_E_CUDA;
    if (cudaFuncSetAttribute(k_compress<false>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)sizeof(CmpSmem)) != cudaSuccess)
        return FASTSGD_E_CUDA;
    if (cudaFuncSetAttribute(k_compress<true>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)sizeof(CmpSmem)) != cudaSuccess)
        return FASTSGD_E_CUDA;
    if (cudaFuncSetAttribute(k_compress<false, true>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)sizeof(CmpSmem)) != cudaSuccess)
        return FASTSGD_E_CUDA;
    if (cudaFuncSetAttribute(k_compress_kv<false>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)sizeof(KvSmem)) != cudaSuccess)
        return FASTSGD_E_CUDA;
    if (cudaFuncSetAttribute(k_compress_kv<true>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)sizeof(KvSmem)) != cudaSuccess)
        return FASTSGD_E_CUDA;
    int b1 = 0, b2 = 0, b3 = 0;
    {
        int b3b = 0;
        if (cudaOccupancyMaxActiveBlocksPerMultiprocessor(&b3, k_compress<false>, kCmpThreads, sizeof(CmpSmem)) != cudaSuccess) return FASTSGD_E_CUDA;
        if (cudaOccupancyMaxActiveBlocksPerMultiprocessor(&b3b, k_compress<true>, kCmpThreads, sizeof(CmpSmem)) != cudaSuccess) return FASTSGD_E_CUDA;
        if (b3b < b3) b3 = b3b;
        if (cudaOccupancyMaxActiveBlocksPerMultiprocessor(&b3b, k_compress<false, true>, kCmpThreads, sizeof(CmpSmem)) != cudaSuccess) return FASTSGD_E_CUDA;
        if (b3b < b3) b3 = b3b;
        int b3c = 0;
        if (cudaOccupancyMaxActiveBlocksPerMultiprocessor(&b3b, k_compress_kv<false>, kKvThreads, sizeof(KvSmem)) != cudaSuccess) return FASTSGD_E_CUDA;
        if (cudaOccupancyMaxActiveBlocksPerMultiprocessor(&b3c, k_compress_kv<true>, kKvThreads, sizeof(KvSmem)) != cudaSuccess) return FASTSGD_E_CUDA;
        g_state.kv_blocks_per_sm = b3b < b3c ? b3b : b3c;
    }
    g_state.cmp_blocks_per_sm = b3;
    if (cudaOccupancyMaxActiveBlocksPerMultiprocessor(&b1, k_abs_sum, kSumThreads, 0) != cudaSuccess) return FASTSGD_E_CUDA;
    if (cudaFuncSetAttribute(k_decode_accumulate<false>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)sizeof(DecShared)) != cudaSuccess)
        return FASTSGD_E_CUDA;
    if (cudaFuncSetAttribute(k_decode_accumulate<true>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)sizeof(DecShared)) != cudaSuccess)
        return FASTSGD_E_CUDA;
    if (cudaFuncSetAttribute(k_decode_accumulate<false, 1>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)sizeof(DecShared)) != cudaSuccess)
        return FASTSGD_E_CUDA;
    if (cudaFuncSetAttribute(k_decode_accumulate<true, 1>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)sizeof(DecShared)) != cudaSuccess)
        return FASTSGD_E_CUDA;
    if (cudaFuncSetAttribute(k_decode_accumulate<false, 2>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)sizeof(DecShared)) != cudaSuccess)
        return FASTSGD_E_CUDA;
    if (cudaFuncSetAttribute(k_decode_accumulate<true, 2>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)sizeof(DecShared)) != cudaSuccess)
        return FASTSGD_E_CUDA;
    if (cudaFuncSetAttribute(k_decode_accumulate<false, 3>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)sizeof(DecShared)) != cudaSuccess)
        return FASTSGD_E_CUDA;
    if (cudaFuncSetAttribute(k_decode_accumulate<true, 3>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)sizeof(DecShared)) != cudaSuccess)
        return FASTSGD_E_CUDA;
    {   // every instantiation must be resident with the grid the launch uses (the queue of large groups relies on it)
        int b2x[8] = {0, 0, 0, 0, 0, 0, 0, 0};
        if (cudaOccupancyMaxActiveBlocksPerMultiprocessor(&b2x[0], k_decode_accumulate<false>, kDecThreads, sizeof(DecShared)) != cudaSuccess) return FASTSGD_E_CUDA;
        if (cudaOccupancyMaxActiveBlocksPerMultiprocessor(&b2x[1], k_decode_accumulate<true>, kDecThreads, sizeof(DecShared)) != cudaSuccess) return FASTSGD_E_CUDA;
        if (cudaOccupancyMaxActiveBlocksPerMultiprocessor(&b2x[2], k_decode_accumulate<false, 1>, kDecThreads, sizeof(DecShared)) != cudaSuccess) return FASTSGD_E_CUDA;
        if (cudaOccupancyMaxActiveBlocksPerMultiprocessor(&b2x[3], k_decode_accumulate<true, 1>, kDecThreads, sizeof(DecShared)) != cudaSuccess) return FASTSGD_E_CUDA;
        if (cudaOccupancyMaxActiveBlocksPerMultiprocessor(&b2x[4], k_decode_accumulate<false, 2>, kDecThreads, sizeof(DecShared)) != cudaSuccess) return FASTSGD_E_CUDA;
        if (cudaOccupancyMaxActiveBlocksPerMultiprocessor(&b2x[5], k_decode_accumulate<true, 2>, kDecThreads, sizeof(DecShared)) != cudaSuccess) return FASTSGD_E_CUDA;
        if (cudaOccupancyMaxActiveBlocksPerMultiprocessor(&b2x[6], k_decode_accumulate<false, 3>, kDecThreads, sizeof(DecShared)) != cudaSuccess) return FASTSGD_E_CUDA;
        if (cudaOccupancyMaxActiveBlocksPerMultiprocessor(&b2x[7], k_decode_accumulate<true, 3>, kDecThreads, sizeof(DecShared)) != cudaSuccess) return FASTSGD_E_CUDA;
        b2 = b2x[0];
        for (int i = 1; i < 8; ++i) if (b2x[i] < b2) b2 = b2x[i];
    }
    g_state.sm_count = sms;
    g_state.sum_blocks_per_sm = b1 > 0 ? b1 : 1;
    g_state.dec_blocks_per_sm = b2 > 0 ? b2 : 1;
    g_state.attrs_set = true;
    return FASTSGD_OK;
}

bool aligned(const void* p, uintptr_t a) { return (reinterpret_cast<uintptr_t>(p) & (a - 1)) == 0; }

int launch_sum(const float* grad, uint64_t n, uint32_t groups, uint32_t tau, const PowTable& pw,
               const WorkspaceView& w, double* sum_out, cudaStream_t st) {
    FSG_DEVICE_STATE();
    SumArgs sa;
    sa.grad = grad; sa.n = n; sa.chunks = (uint32_t)chunks_of(n); sa.groups = groups; sa.tau = tau;
    sa.ctl = w.ctl; sa.thr = w.thr; sa.partials = w.partials; sa.desc = w.desc; sa.sum_out = sum_out;
    uint64_t grid = (uint64_t)g_state.sm_count * g_state.sum_blocks_per_sm;
    if (grid > sa.chunks) grid = sa.chunks;
    { LaunchTimer lt(0, st); k_abs_sum<<<(unsigned)grid, kSumThreads, 0, st>>>(sa, pw); }
    g_launches.fetch_add(1, std::memory_order_relaxed);
    return cudaGetLastError() == cudaSuccess ? FASTSGD_OK : FASTSGD_E_CUDA;
}

}  // namespace

extern "C" {

int fastsgd_version(void) { return 1; }

int fastsgd_kernel_timing_enable(int enable) {
    std::lock_guard<std::mutex> lock(g_mu);
    g_timing = enable != 0;
    return FASTSGD_OK;
}

int fastsgd_kernel_timing_read(double ms_total[3], uint64_t launches[3]) {
    if (!ms_total || !launches) return FASTSGD_E_NULL;
    std::lock_guard<std::mutex> lock(g_mu);
    for (int i = 0; i < 3; ++i) { ms_total[i] = 0.0; launches[i] = 0; }
    int rc = FASTSGD_OK;
    for (const TimedLaunch& t : g_timed) {
        float ms = 0.f;
        if (cudaEventSynchronize(t.stop) != cudaSuccess || cudaEventElapsedTime(&ms, t.start, t.stop) != cudaSuccess) rc = FASTSGD_E_CUDA;
        else { ms_total[t.kernel] += ms; launches[t.kernel] += 1; }
        g_event_pool.emplace_back(t.start, t.stop);
    }
    g_timed.clear();
    return rc;
}

uint64_t fastsgd_launch_count(void) { return g_launches.load(std::memory_order_relaxed); }

int fastsgd_debug_set_wait_limits(uint32_t block_polls, uint32_t copy_tries, uint32_t queue_polls) {
    std::lock_guard<std::mutex> lock(g_mu);
    g_tun.wait_limit = block_polls ? block_polls : kWaitLimit;
    g_tun.try_limit = copy_tries ? copy_tries : kTryLimit;
    g_tun.dec_spin_limit = queue_polls == 0xFFFFFFFFu ? 0u : (queue_polls ? queue_polls : kDecSpinLimit);
    return FASTSGD_OK;
}

int fastsgd_debug_set_grid(uint32_t blocks) {
    std::lock_guard<std::mutex> lock(g_mu);
    g_tun.grid_override = blocks;
    return FASTSGD_OK;
}

int fastsgd_debug_layout(uint64_t* offsets, uint32_t count) {
    if (!offsets) return FASTSGD_E_NULL;
    const uint64_t v[FASTSGD_DEBUG_LAYOUT_FIELDS] = {
        offsetof(Control, bar_count), offsetof(Control, ne_count), offsetof(Control, error),
        kTraceOffset, kJobTraceOffset, kJobTraceBytes, kQueueOffset, offsetof(Control, dq)};
    for (uint32_t i = 0; i < count && i < (uint32_t)FASTSGD_DEBUG_LAYOUT_FIELDS; ++i) offsets[i] = v[i];
    return FASTSGD_OK;
}

int fastsgd_debug_trace_compiled(void) {
#ifdef FASTSGD_TRACE
    return 1;
#else
    return 0;
#endif
}

const char* fastsgd_strerror(int code) {
    switch (code) {
        case FASTSGD_OK: return "ok";
        case FASTSGD_E_NULL: return "null pointer argument";
        case FASTSGD_E_ALIGN: return "pointer not aligned as required";
        case FASTSGD_E_BAD_PARAM: return "invalid parameters";
        case FASTSGD_E_BAD_N: return "n must satisfy 1 <= n < 2^31";
        case FASTSGD_E_CAPACITY: return "output capacity smaller than header + directory";
        case FASTSGD_E_NO_WORKSPACE: return "no workspace registered or workspace too small";
        case FASTSGD_E_NOT_IMPLEMENTED: return "parameter combination not implemented in this build";
        case FASTSGD_E_CUDA: return "CUDA runtime error";
        case FASTSGD_E_TRUNCATED: return "stream shorter than its header";
        case FASTSGD_E_TOO_LARGE: return "n exceeds the built-in scratch of fastsgd_abs_sum_noalloc (2^28 entries)";
        case FASTSGD_ST_NONFINITE: return "sum of |v| is not finite";
        case FASTSGD_ST_CAPACITY: return "stream does not fit in the output buffer";
        case FASTSGD_ST_TIMEOUT: return "bounded wait between thread blocks ran out";
        case FASTSGD_ST_BAD_MAGIC: return "bad magic";
        case FASTSGD_ST_BAD_VERSION: return "bad version";
        case FASTSGD_ST_BAD_STATUS: return "stream carries an error status";
        case FASTSGD_ST_N_MISMATCH: return "n differs from the header";
        case FASTSGD_ST_PARAM_MISMATCH: return "parameters differ from the header";
        case FASTSGD_ST_TRUNCATED: return "stream truncated";
        case FASTSGD_ST_BAD_DIRECTORY: return "inconsistent directory";
        case FASTSGD_ST_BAD_KEY: return "decoded key out of range";
        case FASTSGD_ST_BAD_CODE: return "code byte out of range";
        default: return "unknown code";
    }
}

uint64_t fastsgd_compress_bound(uint64_t n, const fastsgd_params* params) {
    int rc = check_params(params, nullptr);
    if (rc != FASTSGD_OK || n == 0) return 0;
    return bound_bytes(n, params);
}

uint64_t fastsgd_workspace_bytes(uint64_t n, const fastsgd_params* params) {
    int rc = check_params(params, nullptr);
    if (rc != FASTSGD_OK || n == 0) return 0;
    return ws_bytes_for(n, params->group_log2);
}

int fastsgd_set_workspace(void* dev_ptr, uint64_t bytes, void* stream) {
    if (!dev_ptr) return FASTSGD_E_NULL;
    if (!aligned(dev_ptr, 256)) return FASTSGD_E_ALIGN;
    if (bytes < kPartialsOffset) return FASTSGD_E_NO_WORKSPACE;   // control block, tables, trace, decoder queue
    std::lock_guard<std::mutex> lock(g_mu);
    FSG_DEVICE_STATE();
    int rc = ensure_device_setup();
    if (rc) return rc;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    if (cudaMemsetAsync(dev_ptr, 0, kPartialsOffset, st) != cudaSuccess) return FASTSGD_E_CUDA;
    if (cudaMemsetAsync(static_cast<unsigned char*>(dev_ptr) + offsetof(Control, decode_status), 0xFF, 8, st) != cudaSuccess)
        return FASTSGD_E_CUDA;
    g_state.ws = dev_ptr;
    g_state.ws_bytes = bytes;
    g_state.timed_out = false;
    return FASTSGD_OK;
}

int fastsgd_abs_sum(const float* grad, uint64_t n, double* sum_out, void* stream) {
    if (!grad || !sum_out) return FASTSGD_E_NULL;
    if (!aligned(grad, 16) || !aligned(sum_out, 8)) return FASTSGD_E_ALIGN;
    int rc = check_n(n);
    if (rc) return rc;
    std::lock_guard<std::mutex> lock(g_mu);
    FSG_DEVICE_STATE();
    if (!g_state.ws || g_state.ws_bytes < ws_bytes_for(n, kGroupLog2)) return FASTSGD_E_NO_WORKSPACE;
    rc = ensure_device_setup();
    if (rc) return rc;
    PowTable pw;
    for (int k = 0; k <= kMaxTau; ++k) pw.P[k] = 1.0;
    return launch_sum(grad, n, 0u, 0u, pw, view(g_state.ws, n), sum_out, static_cast<cudaStream_t>(stream));
}

namespace {
// The list encoder (kv.cuh).  dense = false: `count` key-value pairs.  dense = true: the gradient `values` of n
// entries itself, read as the list (i, v_i), with its sum already in the workspace.  Caller holds g_state.mu.
int launch_list_encoder(bool dense, const uint32_t* keys, const float* values, uint64_t count, uint64_t n,
                        const fastsgd_params* params, const PowTable& pw, void* out, uint64_t out_bytes, cudaStream_t st,
                        const unsigned long long* count_dev = nullptr, uint32_t run_if = 0u, bool given_sum = false) {
    FSG_DEVICE_STATE();
    if (g_state.kv_blocks_per_sm < 1) return FASTSGD_E_CUDA;
    const uint64_t G = groups_of(n, params->group_log2);
    WorkspaceView w = view(g_state.ws, n, params->group_log2);
    KvArgs ka;
    std::memset(&ka, 0, sizeof(ka));
    ka.keys = keys; ka.vals = values; ka.count = dense ? n : count; ka.n = n;
    ka.out = static_cast<uint8_t*>(out); ka.out_bytes = out_bytes; ka.ctl = w.ctl;
    ka.partials = reinterpret_cast<double*>(static_cast<unsigned char*>(g_state.ws) + kKvPartialsOffset);
    ka.meta = w.desc;
    ka.blk_agg = reinterpret_cast<unsigned long long*>(static_cast<unsigned char*>(g_state.ws) + kKvAggOffset);
    ka.base = params->base; ka.G = (uint32_t)G; ka.chunks = (uint32_t)chunks_of(n);
    ka.tau = params->tau; ka.l = params->flag_bits; ka.group_log2 = params->group_log2;
    ka.wait_limit = g_tun.wait_limit; ka.given_sum = (dense || given_sum) ? 1u : 0u;
    ka.count_dev = count_dev; ka.run_if = run_if;
    // a warp per 32 list entries (dense: per group) until the GPU is full; all blocks are resident: they meet at grid barriers
    const uint64_t units = dense ? G : (count_dev ? n : count);      // (a list made on the device: its length is not known here)
    const uint64_t per_warp = dense ? 1ull : 32ull;
    uint64_t grid = (units + per_warp * kKvWarps - 1) / (per_warp * kKvWarps);
    const uint64_t cap = (uint64_t)g_state.sm_count * (uint64_t)(g_state.kv_blocks_per_sm > 2 ? 2 : g_state.kv_blocks_per_sm);
    if (grid > cap) grid = cap;
    if (grid > kKvMaxGrid) grid = kKvMaxGrid;
    if (g_tun.grid_override && g_tun.grid_override < grid) grid = g_tun.grid_override;
    if (grid < 1) grid = 1;
    const uint64_t warps = grid * kKvWarps;
    uint64_t slice = (units + warps - 1) / warps;
    if (!dense) slice = (slice + 31ull) & ~31ull;
    if (slice < per_warp) slice = per_warp;
    ka.slice = (uint32_t)slice;
    PowTable pwc = pw;
    void* kargs[] = {&ka, &pwc};
    cudaError_t err;
    {
        LaunchTimer lt(1, st);
        err = cudaLaunchCooperativeKernel(dense ? (const void*)k_compress_kv<true> : (const void*)k_compress_kv<false>,
                                          dim3((unsigned)grid), dim3(kKvThreads), kargs, sizeof(KvSmem), st);
    }
    if (err != cudaSuccess) { cudaGetLastError(); return FASTSGD_E_CUDA; }
    g_launches.fetch_add(1, std::memory_order_relaxed);
    return FASTSGD_OK;
}

// The encoder's launches: num_grads dense gradients, up to 8 per launch.
int compress_launches(const float* const* grads, uint64_t n, const fastsgd_params* params,
                      void* const* outs, uint64_t out_bytes, uint32_t num_grads, void* stream) {
    if (!outs || !params || !grads) return FASTSGD_E_NULL;
    for (uint32_t i = 0; i < num_grads; ++i) {
        if (!grads[i] || !outs[i]) return FASTSGD_E_NULL;
        if (!aligned(grads[i], 16) || !aligned(outs[i], 16)) return FASTSGD_E_ALIGN;
    }
    PowTable pw;
    int rc = check_params(params, &pw);
    if (rc) return rc;
    rc = check_n(n);
    if (rc) return rc;
    const uint64_t G = groups_of(n, params->group_log2);
    if (out_bytes < kHeaderBytes + 8ull * G) return FASTSGD_E_CAPACITY;
    if (bound_bytes(n, params) / 4ull >= (1ull << 31)) return FASTSGD_E_BAD_N;   // descriptor fields are 31 bits
    std::lock_guard<std::mutex> lock(g_mu);
    FSG_DEVICE_STATE();
    if (!g_state.ws || g_state.timed_out || g_state.ws_bytes < ws_bytes_for(n, params->group_log2)) return FASTSGD_E_NO_WORKSPACE;
    rc = ensure_device_setup();
    if (rc) return rc;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    if (params->group_log2 != (uint32_t)kGroupLog2) {
        // Any other group size: the sum kernel, then the list encoder over the dense gradient (the fused kernel's
        // tile is the group of 2^14).  Two launches per gradient, the gradient read three times.
        if (params->group_log2 < 8u) return FASTSGD_E_NOT_IMPLEMENTED;
        // sum kernel; the kept entries selected into a list in the workspace (the fused kernel's scratch for dense tiles,
        // 4.5 M pairs); the list encoder on that list -- or, should the list not fit, over the dense gradient itself
        // (a warp per group: slow for large groups).  Which of the two runs is decided on the device.
        unsigned char* wsb = static_cast<unsigned char*>(g_state.ws);
        double* S = reinterpret_cast<double*>(wsb + kJobSumOffset);
        unsigned long long* count_dev = reinterpret_cast<unsigned long long*>(wsb + kKvAggOffset + kKvAggBytes - 8);
        unsigned char* list = wsb + ws_dense_offset(n, params->group_log2);
        const uint64_t capacity = ((uint64_t)kMaxCtas * kDenseScratchBytes) / 8ull;
        for (uint32_t i = 0; i < num_grads; ++i) {
            rc = launch_sum(grads[i], n, 0u, params->tau, pw, view(g_state.ws, n, params->group_log2), S, st);
            if (rc) return rc;
            SelArgs sa;
            std::memset(&sa, 0, sizeof(sa));
            sa.grad = grads[i]; sa.n = n; sa.ctl = reinterpret_cast<Control*>(wsb);
            sa.blk_agg = reinterpret_cast<unsigned long long*>(wsb + kKvAggOffset);
            sa.keys = reinterpret_cast<uint32_t*>(list); sa.vals = reinterpret_cast<float*>(list + 4ull * capacity);
            sa.count_out = count_dev; sa.capacity = capacity; sa.tau = params->tau; sa.wait_limit = g_tun.wait_limit;
            uint64_t sgrid = (uint64_t)g_state.sm_count * 2ull;
            const uint64_t steps = (n + 127ull) >> 7;
            if (sgrid > (steps + kKvWarps - 1) / kKvWarps) sgrid = (steps + kKvWarps - 1) / kKvWarps;
            if (sgrid > 511) sgrid = 511;                      // (one thread per block adds up the totals; the last slot holds the count)
            PowTable pwc = pw;
            void* kargs[] = {&sa, &pwc};
            if (cudaLaunchCooperativeKernel((const void*)k_select_pairs, dim3((unsigned)sgrid), dim3(kKvThreads), kargs, 0, st) != cudaSuccess) {
                cudaGetLastError();
                return FASTSGD_E_CUDA;
            }
            g_launches.fetch_add(1, std::memory_order_relaxed);
            rc = launch_list_encoder(false, sa.keys, sa.vals, 0, n, params, pw, outs[i], out_bytes, st, count_dev, 1u, true);
            if (rc) return rc;
            rc = launch_list_encoder(true, nullptr, grads[i], n, n, params, pw, outs[i], out_bytes, st, count_dev, 2u, true);
            if (rc) return rc;
        }
        return FASTSGD_OK;
    }
    WorkspaceView w = view(g_state.ws, n);
    if (g_state.cmp_blocks_per_sm < 1) return FASTSGD_E_CUDA;
    uint64_t grid = (uint64_t)g_state.sm_count * g_state.cmp_blocks_per_sm;
    if (grid > kMaxCtas) grid = kMaxCtas;
    const uint64_t grid_full = grid;
    if (g_tun.grid_override && g_tun.grid_override < grid) grid = g_tun.grid_override;      // (never two teams then)
    if (grid > G) grid = G;
    for (uint32_t first = 0; first < num_grads; first += kCmpMaxJobs) {
        CmpBatch cb;
        std::memset(&cb, 0, sizeof(cb));
        cb.jobs = num_grads - first < (uint32_t)kCmpMaxJobs ? num_grads - first : (uint32_t)kCmpMaxJobs;
        for (uint32_t i = 0; i < cb.jobs; ++i) {
            cb.grad[i] = grads[first + i];
            cb.out[i] = static_cast<uint8_t*>(outs[first + i]);
        }
        cb.out_bytes = out_bytes; cb.n = n; cb.ctl = w.ctl; cb.partials = w.partials; cb.desc = w.desc; cb.prefix = w.prefix; cb.tmax = w.tmax; cb.nelist = w.nelist; cb.nebits = w.nebits;
        cb.sm_slots = reinterpret_cast<unsigned int*>(static_cast<unsigned char*>(g_state.ws) + kSmSlotOffset);
        cb.dense_scratch = static_cast<unsigned char*>(g_state.ws) + ws_dense_offset(n, params->group_log2);
        cb.base = params->base; cb.G = (uint32_t)G; cb.tau = params->tau; cb.l = params->flag_bits;
        cb.wait_limit = g_tun.wait_limit; cb.try_limit = g_tun.try_limit;
        // Two or more gradients, two resident blocks per SM and enough tiles: the two blocks of an SM
        // form two teams that work on different gradients.  One gradient: the tiles below the grid
        // size are assigned statically, so every block gets an equal share.
        uint64_t launch_grid = grid;
        cb.teams = 1u;
        if (cb.jobs >= 2u && g_state.cmp_blocks_per_sm >= 2 && grid_full == 2ull * (uint64_t)g_state.sm_count &&
            g_state.sm_count <= 256 && G >= grid_full && !g_tun.grid_override) {
            cb.teams = 2u;
            launch_grid = grid_full;
        } else if (cb.jobs == 1u) {
            const uint64_t rounds = (G + grid - 1) / grid;
            launch_grid = (G + rounds - 1) / rounds;
        }
        void* kargs[] = {&cb, &pw};
        cudaError_t err;
        {
            LaunchTimer lt(1, st);
            const void* fn = cb.jobs > 1u ? (const void*)k_compress<true>
                                          : (cb.G > kCmpBigTiles ? (const void*)k_compress<false, true> : (const void*)k_compress<false>);
            err = cudaLaunchCooperativeKernel(fn, dim3((unsigned)launch_grid), dim3(kCmpThreads), kargs, sizeof(CmpSmem), st);
        }
        if (err != cudaSuccess) { cudaGetLastError(); return FASTSGD_E_CUDA; }
        g_launches.fetch_add(1, std::memory_order_relaxed);
    }
    return FASTSGD_OK;
}
}  // namespace

int fastsgd_compress_batch(const float* const* grads, uint64_t n, const fastsgd_params* params,
                           void* const* outs, uint64_t out_bytes, uint32_t num_grads, void* stream) {
    if (!grads) return FASTSGD_E_NULL;
    return compress_launches(grads, n, params, outs, out_bytes, num_grads, stream);
}

int fastsgd_compress_kv(const uint32_t* keys, const float* values, uint64_t count, uint64_t n,
                        const fastsgd_params* params, void* out, uint64_t out_bytes, void* stream) {
    if (!out || !params) return FASTSGD_E_NULL;
    if (count && (!keys || !values)) return FASTSGD_E_NULL;
    if (!aligned(keys, 4) || !aligned(values, 4) || !aligned(out, 16)) return FASTSGD_E_ALIGN;
    PowTable pw;
    int rc = check_params(params, &pw);
    if (rc) return rc;
    rc = check_n(n);
    if (rc) return rc;
    if (count > n) return FASTSGD_E_BAD_N;
    const uint64_t G = groups_of(n, params->group_log2);
    if (out_bytes < kHeaderBytes + 8ull * G) return FASTSGD_E_CAPACITY;
    if (bound_bytes(n, params) / 4ull >= (1ull << 31)) return FASTSGD_E_BAD_N;
    std::lock_guard<std::mutex> lock(g_mu);
    FSG_DEVICE_STATE();
    if (!g_state.ws || g_state.timed_out || g_state.ws_bytes < ws_bytes_for(n, params->group_log2)) return FASTSGD_E_NO_WORKSPACE;
    rc = ensure_device_setup();
    if (rc) return rc;
    return launch_list_encoder(false, keys, values, count, n, params, pw, out, out_bytes, static_cast<cudaStream_t>(stream));
}

int fastsgd_compress(const float* grad, uint64_t n, const fastsgd_params* params,
                     void* out, uint64_t out_bytes, void* stream) {
    if (!grad || !out) return FASTSGD_E_NULL;
    const float* g1[1] = {grad};
    void* o1[1] = {out};
    return fastsgd_compress_batch(g1, n, params, o1, out_bytes, 1u, stream);
}

namespace {
// The decoder's launches over a list of streams, 8 per launch.  adam == nullptr: aggregation into
// dense_out; else the model-update pass (dense_out holds the aggregated gradient), or, `fused` (one
// launch's worth of streams, dense_out all zero), aggregation and update in the same launch.
int decode_launches(const void* const* streams_in, const uint64_t* bytes, uint32_t num_streams, uint64_t n,
                    const fastsgd_params* params, float* dense_out, const fastsgd_adam* adam,
                    float* theta, float* m, float* v, void* stream, bool fused = false, bool packed = false) {
    if (fused && (!adam || num_streams > (uint32_t)kDecMaxStreams)) return FASTSGD_E_BAD_PARAM;
    if (packed && !fused) return FASTSGD_E_BAD_PARAM;
    if (!streams_in || !bytes || !dense_out || !params) return FASTSGD_E_NULL;
    if (!aligned(dense_out, 4)) return FASTSGD_E_ALIGN;
    PowTable pw;
    int rc = check_params(params, &pw);
    if (rc) return rc;
    rc = check_n(n);
    if (rc) return rc;
    // (the queue of groups that whole blocks decode has 2^17 slots)
    if (params->group_log2 < 8u || groups_of(n, params->group_log2) > (kQueueBytes >> 2)) return FASTSGD_E_NOT_IMPLEMENTED;
    for (uint32_t i = 0; i < num_streams; ++i) {
        if (!streams_in[i]) return FASTSGD_E_NULL;
        if (!aligned(streams_in[i], 16)) return FASTSGD_E_ALIGN;
        if (bytes[i] < kHeaderBytes) return FASTSGD_E_TRUNCATED;
    }
    std::lock_guard<std::mutex> lock(g_mu);
    FSG_DEVICE_STATE();
    if (!g_state.ws || g_state.timed_out || g_state.ws_bytes < ws_bytes_for(n, params->group_log2)) return FASTSGD_E_NO_WORKSPACE;
    rc = ensure_device_setup();
    if (rc) return rc;
    const uint64_t G = groups_of(n, params->group_log2);
    // a warp per group at least; for few groups a block per group (up to two per SM), since groups
    // with many keys are decoded by whole blocks taken from a shared queue
    const int warps_per_block = kDecThreads / 32;
    uint64_t grid = (G + warps_per_block - 1) / warps_per_block;
    const uint64_t want = 2ull * (uint64_t)g_state.sm_count;
    const uint64_t per_group = G < want ? G : want;
    if (grid < per_group) grid = per_group;
    const uint64_t cap = (uint64_t)g_state.sm_count * g_state.dec_blocks_per_sm;
    if (grid > cap) grid = cap;
    const uint64_t min_grid = (G + kDecListMax - 1) / kDecListMax;     // a block owns at most kDecListMax groups
    if (grid < min_grid) grid = min_grid;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    for (uint32_t first = 0; first < num_streams; first += kDecMaxStreams) {
        DecArgs da;
        std::memset(&da, 0, sizeof(da));
        da.W = num_streams - first < (uint32_t)kDecMaxStreams ? num_streams - first : (uint32_t)kDecMaxStreams;
        for (uint32_t i = 0; i < da.W; ++i) {
            da.stream[i] = static_cast<const uint8_t*>(streams_in[first + i]);
            da.bytes[i] = bytes[first + i];
        }
        da.n = n; da.dense = dense_out;
        da.status = &view(g_state.ws, n).ctl->decode_status;
        da.trace = reinterpret_cast<unsigned long long*>(static_cast<unsigned char*>(g_state.ws) + kTraceOffset);
        da.q_ctl = view(g_state.ws, n).ctl->dq;
        da.q_list = reinterpret_cast<unsigned int*>(static_cast<unsigned char*>(g_state.ws) + kQueueOffset);
        da.base = params->base; da.G = (uint32_t)G; da.tau = params->tau; da.l = params->flag_bits;
        da.group_log2 = params->group_log2;
        da.spin_limit = g_tun.dec_spin_limit; da.try_limit = g_tun.try_limit;
        if (adam) {
            da.theta = theta; da.m = m; da.v = v;
            da.lr = adam->lr; da.beta1 = adam->beta1; da.beta2 = adam->beta2; da.eps = adam->eps;
        }
        {
            LaunchTimer lt(2, st);
            if (packed) {
                if (da.W == 1u) k_decode_accumulate<true, 3><<<(unsigned)grid, kDecThreads, sizeof(DecShared), st>>>(da, pw);
                else k_decode_accumulate<false, 3><<<(unsigned)grid, kDecThreads, sizeof(DecShared), st>>>(da, pw);
            } else if (fused) {
                if (da.W == 1u) k_decode_accumulate<true, 2><<<(unsigned)grid, kDecThreads, sizeof(DecShared), st>>>(da, pw);
                else k_decode_accumulate<false, 2><<<(unsigned)grid, kDecThreads, sizeof(DecShared), st>>>(da, pw);
            } else if (adam) {
                if (da.W == 1u) k_decode_accumulate<true, 1><<<(unsigned)grid, kDecThreads, sizeof(DecShared), st>>>(da, pw);
                else k_decode_accumulate<false, 1><<<(unsigned)grid, kDecThreads, sizeof(DecShared), st>>>(da, pw);
            } else {
                if (da.W == 1u) k_decode_accumulate<true><<<(unsigned)grid, kDecThreads, sizeof(DecShared), st>>>(da, pw);
                else k_decode_accumulate<false><<<(unsigned)grid, kDecThreads, sizeof(DecShared), st>>>(da, pw);
            }
        }
        g_launches.fetch_add(1, std::memory_order_relaxed);
        if (cudaGetLastError() != cudaSuccess) return FASTSGD_E_CUDA;
    }
    return FASTSGD_OK;
}
}  // namespace

int fastsgd_decompress_accumulate_batch(const void* const* streams_in, const uint64_t* bytes,
                                        uint32_t num_streams, uint64_t n, const fastsgd_params* params,
                                        float* dense_out, void* stream) {
    return decode_launches(streams_in, bytes, num_streams, n, params, dense_out, nullptr, nullptr, nullptr, nullptr, stream);
}

int fastsgd_sparse_adam_update_batch(const void* const* streams_in, const uint64_t* bytes,
                                     uint32_t num_streams, uint64_t n, const fastsgd_params* params,
                                     const fastsgd_adam* hyper, float* grad_scratch,
                                     float* theta, float* m, float* v, void* stream) {
    if (!hyper || !grad_scratch || !theta || !m || !v) return FASTSGD_E_NULL;
    if (!aligned(theta, 4) || !aligned(m, 4) || !aligned(v, 4)) return FASTSGD_E_ALIGN;
    // up to 8 streams: one launch, each group aggregated and its coordinates updated by the warp or block that decodes it
    if (num_streams <= (uint32_t)kDecMaxStreams)
        return decode_launches(streams_in, bytes, num_streams, n, params, grad_scratch, hyper, theta, m, v, stream, true);
    // more: pass 1, the aggregated gradient; pass 2, the same streams again, every key's coordinate updated once
    int rc = decode_launches(streams_in, bytes, num_streams, n, params, grad_scratch, nullptr, nullptr, nullptr, nullptr, stream);
    if (rc) return rc;
    return decode_launches(streams_in, bytes, num_streams, n, params, grad_scratch, hyper, theta, m, v, stream);
}

int fastsgd_sparse_adam_update_packed_batch(const void* const* streams_in, const uint64_t* bytes,
                                            uint32_t num_streams, uint64_t n, const fastsgd_params* params,
                                            const fastsgd_adam* hyper, float* state, void* stream) {
    if (!hyper || !state || !params) return FASTSGD_E_NULL;
    if (!aligned(state, 16)) return FASTSGD_E_ALIGN;
    // (the update of a group lives in the 64 KiB slice of shared memory of the block that decodes it: groups of up to 2^14
    //  indices, one launch's worth of streams)
    if (params->group_log2 > 14u || num_streams > (uint32_t)kDecMaxStreams) return FASTSGD_E_NOT_IMPLEMENTED;
    return decode_launches(streams_in, bytes, num_streams, n, params, state, hyper, nullptr, nullptr, nullptr, stream, true, true);
}

uint64_t fastsgd_key_encode_paper_bound(uint64_t d, uint32_t flag_bits) {
    if (flag_bits < 1 || flag_bits > 5 || d >= (1ull << 31)) return 0;
    const uint64_t blocks = (d + kBkBlockKeys - 1) / kBkBlockKeys;
    const uint64_t words = (d * (flag_bits + 32ull) + 31ull) / 32ull + 1ull;      // widest levels everywhere, and the padding word
    return 16ull + 8ull * blocks + 4ull * words;
}

int fastsgd_key_encode_paper(const uint32_t* keys, uint64_t d, uint32_t flag_bits,
                             void* out, uint64_t out_bytes, void* stream) {
    if (!out || (!keys && d)) return FASTSGD_E_NULL;
    if (!aligned(out, 16) || !aligned(keys, 4)) return FASTSGD_E_ALIGN;
    const uint64_t need = fastsgd_key_encode_paper_bound(d, flag_bits);
    if (!need) return FASTSGD_E_BAD_PARAM;
    if (out_bytes < need) return FASTSGD_E_CAPACITY;
    int sm_count = 0;
    {
        std::lock_guard<std::mutex> lock(g_mu);
        FSG_DEVICE_STATE();
        const int rc = ensure_device_setup();
        if (rc) return rc;
        sm_count = g_state.sm_count;
    }
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    BkArgs a;
    a.keys = keys; a.d = d; a.l = flag_bits;
    a.blocks = (uint32_t)((d + kBkBlockKeys - 1) / kBkBlockKeys);
    a.header = static_cast<uint32_t*>(out);
    a.index = reinterpret_cast<unsigned long long*>(static_cast<unsigned char*>(out) + 16);
    a.bk = reinterpret_cast<uint32_t*>(static_cast<unsigned char*>(out) + 16 + 8ull * a.blocks);
    if (cudaMemsetAsync(out, 0, 16, st) != cudaSuccess) return FASTSGD_E_CUDA;
    if (a.blocks) {
        const unsigned cap = 8u * (unsigned)sm_count;
        const unsigned want = (unsigned)((d + kBkThreads - 1) / kBkThreads);
        k_bk_maxdelta<<<want < cap ? want : cap, kBkThreads, 0, st>>>(a);
        k_bk_sizes<<<a.blocks, kBkThreads, 0, st>>>(a);
    }
    k_bk_scan<<<1, kBkThreads, 0, st>>>(a);
    if (a.blocks) k_bk_pack<<<a.blocks, kBkThreads, 0, st>>>(a);
    g_launches.fetch_add(a.blocks ? 4 : 1, std::memory_order_relaxed);
    if (cudaGetLastError() != cudaSuccess) return FASTSGD_E_CUDA;
    return FASTSGD_OK;
}

int fastsgd_decompress_accumulate(const void* stream_in, uint64_t bytes, uint64_t n,
                                  const fastsgd_params* params, float* dense_out, void* stream) {
    if (!stream_in) return FASTSGD_E_NULL;
    const void* one[1] = {stream_in};
    return fastsgd_decompress_accumulate_batch(one, &bytes, 1u, n, params, dense_out, stream);
}

int fastsgd_stream_info(const void* stream_in, void* stream, uint64_t* total_bytes, uint64_t* d, int* status) {
    if (!stream_in) return FASTSGD_E_NULL;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    unsigned char h[kHeaderBytes];
    if (cudaMemcpyAsync(h, stream_in, kHeaderBytes, cudaMemcpyDeviceToHost, st) != cudaSuccess) return FASTSGD_E_CUDA;
    if (cudaStreamSynchronize(st) != cudaSuccess) return FASTSGD_E_CUDA;
    uint32_t s32; uint64_t v;
    std::memcpy(&s32, h + 8, 4);
    if (status) *status = (int)s32;
    if (s32 == (uint32_t)FASTSGD_ST_TIMEOUT) {        // the launch that wrote this stream left the workspace's counters mid-way
        std::lock_guard<std::mutex> lock(g_mu);
    FSG_DEVICE_STATE();
        g_state.timed_out = true;
    }
    if (d) { std::memcpy(&v, h + 24, 8); *d = v; }
    if (total_bytes) { std::memcpy(&v, h + 32, 8); *total_bytes = v; }
    return FASTSGD_OK;
}

int fastsgd_decode_status(void* stream, int* status) {
    if (!status) return FASTSGD_E_NULL;
    std::lock_guard<std::mutex> lock(g_mu);
    FSG_DEVICE_STATE();
    if (!g_state.ws) return FASTSGD_E_NO_WORKSPACE;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    unsigned long long v = 0;
    unsigned char* p = static_cast<unsigned char*>(g_state.ws) + offsetof(Control, decode_status);
    if (cudaMemcpyAsync(&v, p, 8, cudaMemcpyDeviceToHost, st) != cudaSuccess) return FASTSGD_E_CUDA;
    if (cudaStreamSynchronize(st) != cudaSuccess) return FASTSGD_E_CUDA;
    *status = (v == ~0ull) ? FASTSGD_ST_OK : (int)(v & 0xFFull);
    if (*status == FASTSGD_ST_TIMEOUT) g_state.timed_out = true;
    if (v != ~0ull) {
        if (cudaMemsetAsync(p, 0xFF, 8, st) != cudaSuccess) return FASTSGD_E_CUDA;
        if (cudaStreamSynchronize(st) != cudaSuccess) return FASTSGD_E_CUDA;
    }
    return FASTSGD_OK;
}

uint64_t fastsgd_host_scratch_bytes(uint64_t n, const fastsgd_params* params) {
    const uint64_t b = fastsgd_compress_bound(n, params);
    if (!b) return 0;
    return ((4ull * n + 255ull) & ~255ull) + ((b + 255ull) & ~255ull);
}

int fastsgd_compress_host(const float* grad_host, uint64_t n, const fastsgd_params* params,
                          void* out_host, uint64_t out_bytes, uint64_t* produced, int* status,
                          void* dev_scratch, uint64_t dev_scratch_bytes, void* stream) {
    if (!grad_host || !out_host || !dev_scratch || !params) return FASTSGD_E_NULL;
    if (!aligned(dev_scratch, 16)) return FASTSGD_E_ALIGN;
    const uint64_t need = fastsgd_host_scratch_bytes(n, params);
    if (!need) return FASTSGD_E_BAD_PARAM;
    if (dev_scratch_bytes < need) return FASTSGD_E_NO_WORKSPACE;
    if (out_bytes < kHeaderBytes) return FASTSGD_E_CAPACITY;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    float* dgrad = static_cast<float*>(dev_scratch);
    unsigned char* dout = static_cast<unsigned char*>(dev_scratch) + ((4ull * n + 255ull) & ~255ull);
    const uint64_t bound = fastsgd_compress_bound(n, params);
    const uint64_t cap = out_bytes < bound ? out_bytes : bound;
    if (cudaMemcpyAsync(dgrad, grad_host, 4ull * n, cudaMemcpyHostToDevice, st) != cudaSuccess) return FASTSGD_E_CUDA;
    int rc = fastsgd_compress(dgrad, n, params, dout, cap, stream);
    if (rc) return rc;
    uint64_t total = 0; int hst = 0;
    rc = fastsgd_stream_info(dout, stream, &total, nullptr, &hst);
    if (rc) return rc;
    if (total > cap) return FASTSGD_E_CUDA;
    if (cudaMemcpyAsync(out_host, dout, total, cudaMemcpyDeviceToHost, st) != cudaSuccess) return FASTSGD_E_CUDA;
    if (cudaStreamSynchronize(st) != cudaSuccess) return FASTSGD_E_CUDA;
    if (produced) *produced = total;
    if (status) *status = hst;
    return FASTSGD_OK;
}

int fastsgd_decompress_accumulate_host(const void* const* streams_host, const uint64_t* bytes,
                                       uint32_t num_streams, uint64_t n, const fastsgd_params* params,
                                       float* dense_host, int accumulate, int* status,
                                       void* dev_scratch, uint64_t dev_scratch_bytes, void* stream) {
    if (!streams_host || !bytes || !dense_host || !dev_scratch || !params) return FASTSGD_E_NULL;
    if (!aligned(dev_scratch, 16)) return FASTSGD_E_ALIGN;
    const uint64_t need = fastsgd_host_scratch_bytes(n, params);
    if (!need) return FASTSGD_E_BAD_PARAM;
    const uint64_t dense_bytes = (4ull * n + 255ull) & ~255ull;
    if (dev_scratch_bytes < need) return FASTSGD_E_NO_WORKSPACE;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    float* ddense = static_cast<float*>(dev_scratch);
    unsigned char* dstream = static_cast<unsigned char*>(dev_scratch) + dense_bytes;
    if (accumulate) {
        if (cudaMemcpyAsync(ddense, dense_host, 4ull * n, cudaMemcpyHostToDevice, st) != cudaSuccess) return FASTSGD_E_CUDA;
    } else {
        if (cudaMemsetAsync(ddense, 0, 4ull * n, st) != cudaSuccess) return FASTSGD_E_CUDA;
    }
    // The streams are copied side by side into the staging area (16-byte aligned each) as long as they fit, then decoded
    // by one batched launch per 8; a stream that does not fit beside the others starts a new round (stream order keeps
    // the next round's copies behind this round's launch).
    const uint64_t room = need - dense_bytes;
    uint32_t i = 0;
    while (i < num_streams) {
        std::vector<const void*> ptrs;
        std::vector<uint64_t> sizes;
        uint64_t used = 0;
        while (i < num_streams) {
            if (!streams_host[i]) return FASTSGD_E_NULL;
            if (bytes[i] > room) return FASTSGD_E_NO_WORKSPACE;
            const uint64_t padded = (bytes[i] + 15ull) & ~15ull;
            if (used + padded > room) break;
            if (cudaMemcpyAsync(dstream + used, streams_host[i], bytes[i], cudaMemcpyHostToDevice, st) != cudaSuccess) return FASTSGD_E_CUDA;
            ptrs.push_back(dstream + used);
            sizes.push_back(bytes[i]);
            used += padded;
            ++i;
        }
        int rc2 = fastsgd_decompress_accumulate_batch(ptrs.data(), sizes.data(), (uint32_t)ptrs.size(), n, params, ddense, stream);
        if (rc2) return rc2;
    }
    if (cudaMemcpyAsync(dense_host, ddense, 4ull * n, cudaMemcpyDeviceToHost, st) != cudaSuccess) return FASTSGD_E_CUDA;
    int dst = 0;
    int rc = fastsgd_decode_status(stream, &dst);
    if (rc) return rc;
    if (status) *status = dst;
    return FASTSGD_OK;
}

}  // extern "C"

// ---------------------------------------------------------------------------------------------
// fastsgd_abs_sum_noalloc: the sum kernel with its scratch inside the library image.
//
// Some callers have no way to give the library scratch memory: they may not call cudaMalloc
// (it synchronises the whole device and can fail when memory is tight), they do not own a
// framework allocator, they only receive an input and an output pointer.  For them the
// per-tile partials and the block counter of the sum kernel live in the array below: part of
// the loaded module on every GPU, 256-byte aligned, never allocated and never freed.
//
// In host code the name `g_noalloc_scratch` is only a handle for the symbol, not a device
// address; the address the kernel may use comes from cudaGetSymbolAddress, looked up once
// per device with that device current.
// ---------------------------------------------------------------------------------------------
namespace {

constexpr uint64_t kNoAllocMaxN      = FASTSGD_NOALLOC_MAX_N;                  // 2^28 entries = 1 GiB of fp32
constexpr uint64_t kNoAllocPartials  = kNoAllocMaxN >> fsg::kChunkLog2;        // 16384 fp64 partials
constexpr uint64_t kNoAllocCtlBytes  = 1024;                                   // control block + boundary table
constexpr uint64_t kNoAllocBytes     = kNoAllocCtlBytes + 8ull * kNoAllocPartials;

static __device__ __align__(256) unsigned char g_noalloc_scratch[kNoAllocBytes];

constexpr int kNoAllocMaxDevices = 64;
struct NoAllocDevice {
    unsigned char* scratch = nullptr;     // device address of g_noalloc_scratch on this GPU
    int            grid_cap = 0;          // blocks that fit the GPU at once
};
std::mutex     g_noalloc_mu;
NoAllocDevice  g_noalloc_dev[kNoAllocMaxDevices];

// once per device, with that device current; allocates nothing
int noalloc_setup(int dev, NoAllocDevice** out) {
    if (dev < 0 || dev >= kNoAllocMaxDevices) return FASTSGD_E_CUDA;
    NoAllocDevice& d = g_noalloc_dev[dev];
    if (!d.scratch) {
        void* p = nullptr;
        if (cudaGetSymbolAddress(&p, g_noalloc_scratch) != cudaSuccess || !p) { cudaGetLastError(); return FASTSGD_E_CUDA; }
        int sms = 0, per_sm = 0;
        if (cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess) return FASTSGD_E_CUDA;
        if (cudaOccupancyMaxActiveBlocksPerMultiprocessor(&per_sm, fsg::k_abs_sum, fsg::kSumThreads, 0) != cudaSuccess)
            return FASTSGD_E_CUDA;
        d.grid_cap = sms * (per_sm > 0 ? per_sm : 1);
        d.scratch = static_cast<unsigned char*>(p);
    }
    *out = &d;
    return FASTSGD_OK;
}

}  // namespace

extern "C" int fastsgd_abs_sum_noalloc(const float* grad, uint64_t n, double* sum_out, void* stream) {
    if (!grad || !sum_out) return FASTSGD_E_NULL;
    if (!aligned(grad, 16) || !aligned(sum_out, 8)) return FASTSGD_E_ALIGN;
    if (n == 0) return FASTSGD_E_BAD_N;
    if (n > kNoAllocMaxN) return FASTSGD_E_TOO_LARGE;              // would not fit the built-in scratch
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess) return FASTSGD_E_CUDA;
    std::lock_guard<std::mutex> lock(g_noalloc_mu);
    NoAllocDevice* d = nullptr;
    int rc = noalloc_setup(dev, &d);
    if (rc) return rc;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    // The array keeps the previous call's contents.  Only the block counter has to start at zero
    // (the kernel leaves it at zero, but a call that was cut short might not have): clear the
    // control block on the stream.  Every partial that is read is written first by this call.
    if (cudaMemsetAsync(d->scratch, 0, sizeof(fsg::Control), st) != cudaSuccess) return FASTSGD_E_CUDA;
    fsg::SumArgs sa;
    sa.grad = grad; sa.n = n; sa.chunks = (uint32_t)((n + fsg::kChunk - 1) >> fsg::kChunkLog2);
    sa.groups = 0u; sa.tau = 0u;
    sa.ctl = reinterpret_cast<fsg::Control*>(d->scratch);
    sa.thr = reinterpret_cast<float*>(d->scratch + fsg::kThrOffset);
    sa.partials = reinterpret_cast<double*>(d->scratch + kNoAllocCtlBytes);
    sa.desc = nullptr;
    sa.sum_out = sum_out;
    fsg::PowTable pw;
    for (int k = 0; k <= fsg::kMaxTau; ++k) pw.P[k] = 1.0;
    unsigned grid = (unsigned)d->grid_cap;
    if (grid > sa.chunks) grid = sa.chunks;
    fsg::k_abs_sum<<<grid, fsg::kSumThreads, 0, st>>>(sa, pw);
    g_launches.fetch_add(1, std::memory_order_relaxed);
    return cudaGetLastError() == cudaSuccess ? FASTSGD_OK : FASTSGD_E_CUDA;
}
