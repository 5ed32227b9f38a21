// libfsoftmax: C ABI, argument validation, per-device attribute cache, size-based dispatcher and
// kernel launchers. The interface contract is in include/fsoftmax.h.

#include "../../include/fsoftmax.h"

#include <atomic>
#include <cmath>
#include <cstdio>
#include <cstddef>
#include <cstdlib>
#include <cstring>
#include <initializer_list>
#include <mutex>
#include <type_traits>
#include <unordered_map>

#include "kernels/block_row.cuh"
#include "kernels/common.cuh"
#include "kernels/log_softmax.cuh"
#include "kernels/norm_row.cuh"
#include "kernels/router_topk.cuh"
#include "kernels/smem_row.cuh"
#include "kernels/softmax_backward.cuh"
#include "kernels/softmax_masked.cuh"
#include "kernels/softmax_split.cuh"
#include "kernels/warp_row.cuh"

namespace {

using namespace fsm;

constexpr int kMaxDevices = 64;
constexpr double kLog2e = 1.4426950408889634074;

thread_local int t_last_cuda_error = 0;

int cuda_fail(cudaError_t e) {
    t_last_cuda_error = static_cast<int>(e);
    (void)cudaGetLastError();   // clear the sticky-free error state
    return FS_ERR_CUDA;
}

#define FS_CUDA(call)                                   \
    do {                                                \
        cudaError_t e__ = (call);                       \
        if (e__ != cudaSuccess) return cuda_fail(e__);  \
    } while (0)

// ---------------------------------------------------------------------------------------------
// per-device state
// ---------------------------------------------------------------------------------------------

struct LaunchInfo {      // cached per (kernel function, threads, dynamic smem, cluster size)
    int blocks_per_sm;   // or active clusters for cluster launches
};

struct Device {
    std::atomic<bool> ready{false};   // set last, with release order, once the fields below are valid
    int sm_count = 0;
    int smem_optin = 0;      // max dynamic shared memory per block
    int cluster_ok = 0;
    int* status = nullptr;   // device status word
    std::atomic<int> wait_polls{kDefaultWaitPolls};   // poll cap handed to the split-row kernel (lowered by the self-test only)
    // scratch of the two-kernel paths (rows beyond a cluster's shared memory): grown on demand, kept,
    // handed from call to call in stream order through scratch_ev, freed by fs_release
    void* scratch = nullptr;
    size_t scratch_bytes = 0;
    cudaEvent_t scratch_ev = nullptr;
    bool scratch_used = false;
    std::unordered_map<uint64_t, LaunchInfo> launch_cache;
    std::unordered_map<const void*, bool> configured;   // kernels whose function attributes are set
    // fs_softmax_host staging
    static constexpr int kSlots = 4;
    cudaStream_t s_in = nullptr, s_run = nullptr, s_out = nullptr;   // copy-in, kernels, copy-out
    cudaEvent_t ev_in[kSlots] = {}, ev_run[kSlots] = {}, ev_out[kSlots] = {};
    void* dx[kSlots] = {};
    void* dy[kSlots] = {};
    size_t slot_bytes = 0;
};

Device g_dev[kMaxDevices];
std::mutex g_mu;          // guards g_dev[*].ready transitions and launch caches
std::mutex g_host_mu;     // serialises fs_softmax_host / fs_release
std::mutex g_scratch_mu;  // serialises the users of Device::scratch from acquire to event record

// Environment switches, each read once per process.
//   FS_LOG=1             one line per call on stderr: the dispatcher's decision and launch geometry
//   FS_FORCE_KERNEL=name the kernel fs_softmax's dispatcher picks (warp, block, block_tma, cluster,
//                        generic); a shape the forced kernel cannot run returns FS_ERR_UNSUPPORTED
//   FS_CHECK=1           slow argument validation: every tensor pointer must be device-accessible
//                        memory of the current device (cudaPointerGetAttributes)
//   FS_SIM_NO_CLUSTER=1  behave as on a device without cluster launch (downgrade paths, tests)
//   FS_SIM_SMEM_OPTIN=n  behave as on a device with n bytes of opt-in shared memory per block
int env_int(const char* name, int dflt) {
    const char* e = std::getenv(name);
    return e && e[0] ? std::atoi(e) : dflt;
}
bool early_prefetch_enabled() { static const bool v = env_int("FS_EARLY_PF", 1) != 0; return v; }
bool wide_store_enabled() { static const bool v = env_int("FS_WIDE_STORE", 1) != 0; return v; }
bool shift_enabled() { static const bool v = env_int("FS_SHIFT", 1) != 0; return v; }
bool log_enabled() { static const bool v = env_int("FS_LOG", 0) != 0; return v; }
bool check_enabled() { static const bool v = env_int("FS_CHECK", 0) != 0; return v; }
#define FS_LOGF(...) do { if (log_enabled()) { std::fprintf(stderr, "[fsoftmax] " __VA_ARGS__); std::fputc('\n', stderr); } } while (0)

int get_device(Device** out) {
    int d = 0;
    FS_CUDA(cudaGetDevice(&d));
    if (d < 0 || d >= kMaxDevices) return FS_ERR_UNSUPPORTED;
    Device& dev = g_dev[d];
    if (!dev.ready.load(std::memory_order_acquire)) {
        std::lock_guard<std::mutex> lk(g_mu);
        if (!dev.ready.load(std::memory_order_relaxed)) {
            FS_CUDA(cudaDeviceGetAttribute(&dev.sm_count, cudaDevAttrMultiProcessorCount, d));
            FS_CUDA(cudaDeviceGetAttribute(&dev.smem_optin, cudaDevAttrMaxSharedMemoryPerBlockOptin, d));
            FS_CUDA(cudaDeviceGetAttribute(&dev.cluster_ok, cudaDevAttrClusterLaunch, d));
            if (env_int("FS_SIM_NO_CLUSTER", 0)) dev.cluster_ok = 0;
            const int sim_smem = env_int("FS_SIM_SMEM_OPTIN", 0);
            if (sim_smem > 0) dev.smem_optin = std::min(dev.smem_optin, std::max(sim_smem, 16 * 1024));
            FS_CUDA(cudaMalloc(&dev.status, sizeof(int)));
            FS_CUDA(cudaMemset(dev.status, 0, sizeof(int)));
            FS_LOGF("device %d: %d SMs, %d B opt-in shared memory per block, cluster launch %s", d, dev.sm_count,
                    dev.smem_optin, dev.cluster_ok ? "yes" : "no");
            dev.ready.store(true, std::memory_order_release);
        }
    }
    *out = &dev;
    return FS_OK;
}

int elem_size(int dtype) { return dtype == FS_DTYPE_FP32 ? 4 : 2; }

// Grid policy: one block (or cluster) per unit of work, handed out by the hardware block scheduler.
// Measured on B200, a plain copy written that way runs ~10% faster than the same copy with one
// resident block per slot looping over a fixed share of the data, because the scheduler balances
// SMs that see different memory latencies; the resident-grid forms of these kernels lost the same way.

// ---------------------------------------------------------------------------------------------
// shape -> kernel geometry (pure host arithmetic, no CUDA calls)
// ---------------------------------------------------------------------------------------------

int next_pow2(int64_t v) { int p = 1; while (p < v) p <<= 1; return p; }

// Largest vectors-per-thread the register budget allows: 64 floats of payload.
int max_vpt(int dtype) { return dtype == FS_DTYPE_FP32 ? 16 : 8; }
int max_threads_for(int dtype, int vpt) { return vpt * (dtype == FS_DTYPE_FP32 ? 4 : 8) <= 16 ? 1024 : 512; }

// Row sizes (bytes) at which the dispatcher changes kernel, from sweeps on B200 (256 MiB of
// traffic per launch, rows from 2 KiB to 1 MiB, every kernel x threads x cluster size, against a
// plain copy of the same bytes).
//   16-bit: (sub-)warp per row up to 4 KiB; above that up to 14 KiB four rows per block, each in
//           shared memory under one warp (softmax_tile_wanted), except 6 and 8 KiB rows, which the
//           block-per-row kernel (direct loads) fits exactly; then the shared-memory-resident split.
//   fp32:   (sub-)warp per row up to 3 KiB, block per row up to 8 KiB, block per row fed by bulk
//           copies up to 32 KiB, then the split.
//   split:  slices of about 32 KiB, cluster and block size chosen per row length (smem_geom);
//           rows beyond 16 x 32 KiB grow the slice.
int64_t warp_max_row_bytes(int dtype) { return dtype == FS_DTYPE_FP32 ? 3072 : 4096; }
int64_t block_max_row_bytes(int) { return 8192; }
constexpr int64_t kSpanMaxRowBytes = 512;
// rows up to this size that are not a multiple of 16 bytes stay with the shifted block kernel; longer ones go to the
// shifted split-row kernel where the device has cluster launch (FS_SHIFT_BLOCK_MAX overrides, bytes). Measured on
// B200, block / split-row: fp32 rows of 4 KB 32.7 / 54.2 us, bf16 rows of 8 KB 75.7 / 76.8, of 24 KB 208 / 70.5, of 60 KB 228 / 97.
int64_t shift_block_max_row_bytes() { static const int64_t v = env_int("FS_SHIFT_BLOCK_MAX", 8192); return v; }            // span_rows_kernel: 128 such rows in a block's shared memory
int64_t block_tma_max_row_bytes(int dtype) { return dtype == FS_DTYPE_FP32 ? 32768 : 0; }

// 16-bit rows the dispatcher gives the four-rows-per-block kernel (softmax_tile_kernel), in 16-byte vectors
// (lo < vectors <= hi): rows above 4 KiB up to 14 KiB, except the two lengths the block-per-row kernel fits
// exactly. Measured on B200 (bf16, 256 MiB per direction, a copy = 80.1 us): 4.5 / 5 / 7 / 9 / 10 / 11 / 12 / 13 / 14 KiB
// rows 81.5 / 81.5 / 81.4 / 81.9 / 81.5 / 81.9 / 81.8 / 82.2 / 84.2 us against 88.1 / 83.8 / 82.6 / 99.7 / 94.0 / 90.9 / 85.7 /
// 93.4 / 88.5 for the block-per-row kernel (up to 8 KiB) and the split-row kernel (beyond); 6 and 8 KiB rows stay
// with the block kernel (79.4 / 79.1 against 81.8 / 81.4), 16 KiB with the split-row kernel (81.2 against 82.8).
// FS_SOFTMAX_TILE "lo:hi" (read once) overrides the range, "0" turns the kernel off.
bool softmax_tile_wanted(int dtype, int64_t nvec) {
    static const std::pair<int64_t, int64_t> ov = [] {
        const char* e = std::getenv("FS_SOFTMAX_TILE");
        if (!e) return std::pair<int64_t, int64_t>(-1, -1);
        long lo = 0, hi = 0;
        if (std::sscanf(e, "%ld:%ld", &lo, &hi) == 2) return std::pair<int64_t, int64_t>(lo, hi);
        return std::pair<int64_t, int64_t>(0, 0);
    }();
    if (dtype == FS_DTYPE_FP32) return false;
    if (ov.first >= 0) return nvec > ov.first && nvec <= ov.second;
    return nvec > 256 && nvec <= 896 && nvec != 384 && nvec != 512;
}
int64_t split_slice_bytes(int) { return 32768; }
constexpr int kMaxCluster = 16;
constexpr int kSplitThreads = 256;                   // block size of the two-kernel (segment) path

int64_t warp_capacity_vecs(int dtype) { return 32 * int64_t(max_vpt(dtype)); }

struct WarpGeom { int lanes, vpl, r; };
// Four vectors per lane where the row allows it (few shuffle steps per element, four loads in
// flight per lane), more lanes per row as rows grow, then more vectors per lane.
bool warp_geom(int64_t nvec, int dtype, WarpGeom* g) {
    if (nvec < 1 || nvec > warp_capacity_vecs(dtype)) return false;
    if (nvec <= 2) { g->lanes = 1; g->vpl = static_cast<int>(nvec); g->r = 4 / g->vpl; return true; }
    g->lanes = std::min(32, next_pow2((nvec + 3) / 4));
    g->vpl = std::max(4, next_pow2((nvec + g->lanes - 1) / g->lanes));
    g->r = 1;
    return true;
}

struct BlockGeom { int threads, vpt; };
// threads == 0: choose. Otherwise honour the forced thread count.
bool block_geom(int64_t nvec, int dtype, int threads, BlockGeom* g) {
    if (nvec < 1) return false;
    const int mv = max_vpt(dtype);
    if (threads > 0) {
        if (threads % 32 || threads > 1024) return false;
        const int vpt = next_pow2((nvec + threads - 1) / threads);
        if (vpt > mv || threads > max_threads_for(dtype, vpt)) return false;
        g->threads = threads; g->vpt = vpt;
        return true;
    }
    // at least two loads in flight per thread, 128-thread blocks until the row outgrows them
    int vpt = 2;
    while (vpt < mv && nvec > 128 * int64_t(vpt)) vpt <<= 1;
    int64_t t = (nvec + vpt - 1) / vpt;
    t = (t + 31) / 32 * 32;
    if (t > max_threads_for(dtype, vpt)) return false;
    g->threads = static_cast<int>(t); g->vpt = vpt;
    return true;
}

// Shared-memory-resident split: which cluster size and block size a row gets.
//
// What decides the speed of this kernel is how many bytes of rows an SM holds at a time (blocks per
// SM x slice), because a block loads, computes and stores one after the other and only the other
// blocks on the SM keep the memory system busy meanwhile. Measured on B200 over rows from 12 KiB
// to 1.5 MiB, every cluster size 1..16 and block sizes 64..256: the best geometry has slices of
// 32 KiB or a little less that are a whole number of chunks (a chunk = 8 vectors per thread, so
// the block size is chosen to divide the slice), two or three chunks per block, and the smallest
// cluster that gets there; cluster sizes need not be powers of two. The candidates are scored by a
// small model of those measurements (mean loss against the best measured geometry: 0.5%).
struct SmemGeom { int cs, slice, threads; };
constexpr int64_t kSmemSliceMaxBytes = 192 * 1024;
constexpr int kSmemPerSm = 228 * 1024;               // shared memory of one SM, 1 KiB reserved per block
constexpr int kSplitThreadsPerSm = 768;              // the split-row kernel's register cap: 85 per thread

bool smem_geom_fits(int64_t nvec, int dtype, int t, int cs, SmemGeom* g) {
    if (cs < 1 || cs > kMaxCluster || t < 32 || t % 32 || t > 256) return false;
    const int64_t slice = (nvec + cs - 1) / cs;
    if (slice * 16 > kSmemSliceMaxBytes) return false;
    if (slice > int64_t(kSmemRowMaxChunks) * smem_row_u(dtype) * t) return false;
    g->cs = cs; g->slice = static_cast<int>(slice); g->threads = t;
    return true;
}

double smem_geom_score(int64_t nvec, int dtype, const SmemGeom& g) {
    const int64_t chunk = int64_t(smem_row_u(dtype)) * g.threads;
    const int64_t nch = (g.slice + chunk - 1) / chunk;
    const bool full = nvec == int64_t(g.slice) * g.cs && g.slice % chunk == 0;
    const double stage = double(nch * chunk * 16);
    // dynamic part + the kernel's static shared memory (896 B) + the 1 KiB the hardware reserves per block
    const double smem = stage + smem_row_tail_bytes(g.threads, int(nch)) + 896 + 1024;
    const int blocks = std::min(std::min(int(kSmemPerSm / smem), kSplitThreadsPerSm / g.threads), 32);
    if (blocks < 1) return 0.0;
    const double resident_cap = 184.0 * 1024;
    double s = std::min(double(blocks) * g.slice * 16, resident_cap) / resident_cap;
    if (!full) s *= 0.93 * (g.slice * 16 / stage);           // bounds checks, arithmetic on the padding
    if (nch == 1) s *= 0.92;                                 // nothing to overlap inside the block
    if (nch > 3) s *= 1.0 - 0.02 * double(nch - 3);
    const double warps = blocks * g.threads / 32.0;
    if (warps < 16.0) s *= 1.0 - (dtype == FS_DTYPE_FP32 ? 0.075 : 0.25) * (1.0 - warps / 16.0);
    // large clusters leave block slots of a GPC unused
    s *= g.cs <= 4 ? 1.0 : g.cs <= 8 ? 0.97 : g.cs <= 12 ? 0.93 : 0.9;
    return s;
}

// threads / cluster == 0: choose. Forced values are honoured (threads a multiple of 32 up to 256,
// cluster 1..16).
bool smem_geom(int64_t nvec, int dtype, int threads, int cluster, SmemGeom* g) {
    if (nvec < 1) return false;
    const int cs_fit = static_cast<int>(std::min<int64_t>(kMaxCluster, (nvec * 16 + split_slice_bytes(dtype) - 1) / split_slice_bytes(dtype)));
    const int cs_lo = cluster ? cluster : (cs_fit < kMaxCluster ? std::max(1, cs_fit - 1) : kMaxCluster);
    const int cs_hi = cluster ? cluster : std::min(kMaxCluster, cs_fit + 1);
    static const int kThreads[] = {128, 96, 160, 192, 256};     // in order of preference
    double best = 0.0;
    bool found = false;
    // cluster sizes nearest the 32 KiB fit first; a later candidate must be 1% better to win
    for (int d = 0; d <= 2; ++d) {
        for (int sgn = 0; sgn < (d ? 2 : 1); ++sgn) {
            const int cs = cluster ? cluster : cs_fit + (sgn ? d : -d);
            if (cs < cs_lo || cs > cs_hi || (cluster && d)) continue;
            for (int ti = 0; ti < (threads ? 1 : 5); ++ti) {
                SmemGeom c;
                if (!smem_geom_fits(nvec, dtype, threads ? threads : kThreads[ti], cs, &c)) continue;
                const double sc = std::max(smem_geom_score(nvec, dtype, c), 1e-9);
                if (!found || sc > best * 1.01) { best = sc; *g = c; found = true; }
            }
        }
    }
    if (!found && !threads) {
        // short slices: fewer threads than the preferred sizes
        for (int t = 64; t >= 32 && !found; t -= 32)
            for (int cs = cs_lo; cs <= cs_hi && !found; ++cs) found = smem_geom_fits(nvec, dtype, t, cs, g);
    }
    return found;
}

bool fast_path_ok(int64_t cols, int dtype, int x_align, int y_align) {
    return x_align >= 16 && y_align >= 16 && (cols * elem_size(dtype)) % 16 == 0;
}

int select_kernel(int64_t cols, int dtype, int x_align, int y_align) {
    if (!fast_path_ok(cols, dtype, x_align, y_align)) return FS_KERNEL_GENERIC;
    const int64_t row_bytes = cols * elem_size(dtype);
    const int64_t nvec = row_bytes / 16;
    WarpGeom wg; BlockGeom bg;
    if (row_bytes <= warp_max_row_bytes(dtype) && warp_geom(nvec, dtype, &wg)) return FS_KERNEL_WARP;
    if (softmax_tile_wanted(dtype, nvec)) return FS_KERNEL_BLOCK_TMA;        // four rows per block, a warp per row
    if (row_bytes <= block_max_row_bytes(dtype) && block_geom(nvec, dtype, 0, &bg)) return FS_KERNEL_BLOCK;
    if (row_bytes <= block_tma_max_row_bytes(dtype) && block_geom(nvec, dtype, 0, &bg)) return FS_KERNEL_BLOCK_TMA;
    SmemGeom sg;
    if (smem_geom(nvec, dtype, 0, 0, &sg)) return FS_KERNEL_CLUSTER;
    return FS_KERNEL_GENERIC;
}

int ptr_align(const void* p) {
    const uintptr_t a = reinterpret_cast<uintptr_t>(p);
    int al = 1;
    while (al < 16 && (a % (al * 2)) == 0) al <<= 1;
    return al;
}

// ---------------------------------------------------------------------------------------------
// launch helpers
// ---------------------------------------------------------------------------------------------

uint64_t cache_key(const void* fn, int threads, size_t smem, int cs) {
    uint64_t h = reinterpret_cast<uintptr_t>(fn);
    h = h * 0x9E3779B97F4A7C15ull ^ (uint64_t(threads) << 40) ^ (uint64_t(smem) << 8) ^ uint64_t(cs);
    return h;
}

// Function attributes are per kernel, not per launch geometry: raise the dynamic shared memory
// limit to the device maximum (never lower it again) and allow cluster sizes above 8, once.
int configure_kernel(Device& dev, const void* fn, bool uses_dynamic_smem, bool is_cluster) {
    {
        std::lock_guard<std::mutex> lk(g_mu);
        if (dev.configured.count(fn)) return FS_OK;
    }
    if (uses_dynamic_smem) {
        cudaFuncAttributes fa;
        FS_CUDA(cudaFuncGetAttributes(&fa, fn));
        const int dyn_max = dev.smem_optin - static_cast<int>(fa.sharedSizeBytes);   // static + dynamic <= opt-in limit
        FS_CUDA(cudaFuncSetAttribute(fn, cudaFuncAttributeMaxDynamicSharedMemorySize, dyn_max));
    }
    if (is_cluster) FS_CUDA(cudaFuncSetAttribute(fn, cudaFuncAttributeNonPortableClusterSizeAllowed, 1));
    std::lock_guard<std::mutex> lk(g_mu);
    dev.configured[fn] = true;
    return FS_OK;
}

// Resident blocks per SM for a kernel at (threads, smem).
int blocks_per_sm(Device& dev, const void* fn, int threads, size_t smem, int* out) {
    const uint64_t key = cache_key(fn, threads, smem, 0);
    {
        std::lock_guard<std::mutex> lk(g_mu);
        auto it = dev.launch_cache.find(key);
        if (it != dev.launch_cache.end()) { *out = it->second.blocks_per_sm; return FS_OK; }
    }
    int rc = configure_kernel(dev, fn, smem > 0, false);
    if (rc != FS_OK) return rc;
    int n = 0;
    FS_CUDA(cudaOccupancyMaxActiveBlocksPerMultiprocessor(&n, fn, threads, smem));
    if (n < 1) return FS_ERR_UNSUPPORTED;
    std::lock_guard<std::mutex> lk(g_mu);
    dev.launch_cache[key] = LaunchInfo{n};
    *out = n;
    return FS_OK;
}

int active_clusters(Device& dev, const void* fn, int threads, size_t smem, int cs, int* out) {
    const uint64_t key = cache_key(fn, threads, smem, cs);
    {
        std::lock_guard<std::mutex> lk(g_mu);
        auto it = dev.launch_cache.find(key);
        if (it != dev.launch_cache.end()) { *out = it->second.blocks_per_sm; return FS_OK; }
    }
    int rc = configure_kernel(dev, fn, true, true);
    if (rc != FS_OK) return rc;
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3(cs * dev.sm_count, 1, 1);
    cfg.blockDim = dim3(threads, 1, 1);
    cfg.dynamicSmemBytes = smem;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeClusterDimension;
    attr[0].val.clusterDim.x = cs; attr[0].val.clusterDim.y = 1; attr[0].val.clusterDim.z = 1;
    cfg.attrs = attr; cfg.numAttrs = 1;
    int n = 0;
    FS_CUDA(cudaOccupancyMaxActiveClusters(&n, fn, &cfg));
    if (n < 1) return FS_ERR_UNSUPPORTED;
    std::lock_guard<std::mutex> lk(g_mu);
    dev.launch_cache[key] = LaunchInfo{n};
    *out = n;
    return FS_OK;
}

// One-shot grids of the split-row and block-per-row kernels: a cluster (block) asks L2 for the
// input of the row that starts about a third of a generation of resident clusters later, so that
// DRAM reads run ahead of the blocks that consume them and no longer pause while a block computes.
// Measured on B200 (384 MiB of bf16 and fp32 rows from 6 KiB to 1 MiB): a quarter to a half of a
// generation brings 6 KiB..512 KiB rows to the speed of a plain copy (before: 0.85-0.98 of it); a
// whole generation is too early (up to 20% slower than none: the lines are gone again before they
// are used), an eighth too late; half costs 2% on 4 GiB of 128 KiB rows, a third does not.
// FS_PREFETCH_PCT (read once) sets the distance in percent of a generation, 0 turns it off.
int64_t prefetch_rows(int resident_clusters) {
    static const int pct = [] { const char* e = std::getenv("FS_PREFETCH_PCT"); return e ? std::max(0, std::atoi(e)) : 30; }();
    return pct == 0 ? 0 : std::max<int64_t>(1, int64_t(resident_clusters) * pct / 100);
}

// The lag between the clusters of a one-shot grid's first wave (first_wave_lag in common.cuh):
// the bytes one cluster loads, at FS_LAG_BW bytes per microsecond (read once; default 6500, this
// part's copy bandwidth; 0 turns the lag off). Measured on B200, 256 rows of 512 KiB bf16: 49.2 us
// without, 47.2-47.4 with a spread of 3-4 us over the 45 resident clusters (5900-7900 bytes/us),
// 47.7-48.1 at half or twice that; orders other than the linear one gain less.
template <class P>
void set_first_wave_lag(P& p, int resident_clusters, int64_t bytes_per_cluster) {
    static const int bw = [] { const char* e = std::getenv("FS_LAG_BW"); return e ? std::max(0, std::atoi(e)) : 6500; }();
    p.lag_rows = resident_clusters;
    p.lag_ns = bw > 0 ? static_cast<float>(double(bytes_per_cluster) / double(bw)) : 0.0f;
    p.early_pf = early_prefetch_enabled();
}

// Programmatic dependent launch (on unless FS_PDL=0): the kernel may be scheduled while the
// previous kernel of the stream drains; it waits (griddepcontrol.wait) before touching memory.
bool pdl_enabled() {
    static const bool v = [] { const char* e = std::getenv("FS_PDL"); return !(e && e[0] == '0'); }();
    return v;
}

// Checked build (-DFS_DEBUG_BOUNDS): the entry points register the address ranges of their tensors,
// every launch uploads them (with the device's status word) to the table the access helpers consult.
// One table per device image: launches from several host threads or streams at once would overwrite
// each other's ranges, so the checked library is for single-stream debugging runs.
struct TensorRange { const void* p; unsigned long long bytes; int writable; };
#ifdef FS_DEBUG_BOUNDS
thread_local DebugRanges t_dbg = {};
thread_local long long t_dbg_shrink = 0;          // self-test: the writable ranges end this many bytes early
void dbg_register(std::initializer_list<TensorRange> ranges) {
    t_dbg = DebugRanges{};
    for (const TensorRange& r : ranges) {
        if (!r.p || t_dbg.n >= 8) continue;
        const unsigned long long lo = reinterpret_cast<unsigned long long>(r.p);
        unsigned long long hi = lo + r.bytes;
        if (r.writable && t_dbg_shrink > 0) hi -= std::min<unsigned long long>(r.bytes, static_cast<unsigned long long>(t_dbg_shrink));
        t_dbg.lo[t_dbg.n] = lo; t_dbg.hi[t_dbg.n] = hi; t_dbg.writable[t_dbg.n] = r.writable;
        ++t_dbg.n;
    }
}
#define FS_DBG_RANGES(...) dbg_register({__VA_ARGS__})
#else
#define FS_DBG_RANGES(...) do { } while (0)
#endif

template <typename... Args>
int launch(const void* fn, int64_t grid, int threads, size_t smem, int cs, cudaStream_t st, Args... args) {
#ifdef FS_DEBUG_BOUNDS
    {   // the ranges only: the flag word and the first refused address stay as the device has them
        cudaStreamCaptureStatus cap = cudaStreamCaptureStatusNone;
        FS_CUDA(cudaStreamIsCapturing(st, &cap));
        // inside a stream capture the copy becomes a graph node that reads its source at every replay: the source
        // must outlive the graph, so it is a small heap block that is never freed (checked build only)
        const DebugRanges* src = cap == cudaStreamCaptureStatusNone ? &t_dbg : new DebugRanges(t_dbg);
        FS_CUDA(cudaMemcpyToSymbolAsync(g_dbg, src, offsetof(DebugRanges, flags), 0, cudaMemcpyHostToDevice, st));
    }
#endif
    void* argv[] = {static_cast<void*>(&args)...};
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3(static_cast<unsigned>(grid), 1, 1);
    cfg.blockDim = dim3(threads, 1, 1);
    cfg.dynamicSmemBytes = smem;
    cfg.stream = st;
    cudaLaunchAttribute attr[2];
    unsigned n = 0;
    if (cs > 0) {
        attr[n].id = cudaLaunchAttributeClusterDimension;
        attr[n].val.clusterDim.x = cs; attr[n].val.clusterDim.y = 1; attr[n].val.clusterDim.z = 1;
        ++n;
    }
    if (pdl_enabled()) {
        attr[n].id = cudaLaunchAttributeProgrammaticStreamSerialization;
        attr[n].val.programmaticStreamSerializationAllowed = 1;
        ++n;
    }
    cfg.attrs = n ? attr : nullptr; cfg.numAttrs = n;
    FS_CUDA(cudaLaunchKernelExC(&cfg, fn, argv));
    return FS_OK;
}

// ---- per-device scratch of the two-kernel paths ----------------------------------------------
// The caller holds g_scratch_mu from scratch_acquire until scratch_done. The buffer is allocated on
// first need and grown (never shrunk) when a call needs more; a call that fits allocates nothing.
// Successive users are ordered on the device by an event: the next user's stream waits for the
// previous user's last kernel. Inside a stream capture no event is waited for or recorded (the
// captured work is ordered by the capture itself) and the buffer cannot grow: such a call returns
// FS_ERR_UNSUPPORTED unless an earlier call outside the capture has already sized the buffer.
int scratch_acquire(Device& dev, size_t bytes, cudaStream_t st, void** out, bool* capturing) {
    cudaStreamCaptureStatus cap = cudaStreamCaptureStatusNone;
    FS_CUDA(cudaStreamIsCapturing(st, &cap));
    *capturing = cap != cudaStreamCaptureStatusNone;
    if (bytes > dev.scratch_bytes) {
        if (*capturing) return FS_ERR_UNSUPPORTED;
        if (dev.scratch) {
            FS_CUDA(cudaDeviceSynchronize());          // earlier users have finished with the old buffer
            FS_CUDA(cudaFree(dev.scratch));
            dev.scratch = nullptr; dev.scratch_bytes = 0; dev.scratch_used = false;
        }
        const size_t want = (std::max<size_t>(bytes, size_t(1) << 20) + 0xfffff) & ~size_t(0xfffff);
        FS_CUDA(cudaMalloc(&dev.scratch, want));
        dev.scratch_bytes = want;
        FS_LOGF("scratch buffer grown to %zu bytes", want);
        if (!dev.scratch_ev) FS_CUDA(cudaEventCreateWithFlags(&dev.scratch_ev, cudaEventDisableTiming));
    } else if (!*capturing && dev.scratch_used) {
        FS_CUDA(cudaStreamWaitEvent(st, dev.scratch_ev, 0));
    }
    *out = dev.scratch;
    return FS_OK;
}

int scratch_done(Device& dev, cudaStream_t st, bool capturing) {
    if (capturing) return FS_OK;
    FS_CUDA(cudaEventRecord(dev.scratch_ev, st));
    dev.scratch_used = true;
    return FS_OK;
}

// ---- kernel tables --------------------------------------------------------------------------

template <int DT, bool NEG> const void* warp_fn(const WarpGeom& g) {
    if (g.vpl == 1) return (const void*)warp_row_kernel<DT, NEG, 1, 1, 4>;
    if (g.vpl == 2) return (const void*)warp_row_kernel<DT, NEG, 1, 2, 2>;
    if (g.vpl == 4) {
        switch (g.lanes) {
            case 1:  return (const void*)warp_row_kernel<DT, NEG, 1, 4, 1>;
            case 2:  return (const void*)warp_row_kernel<DT, NEG, 2, 4, 1>;
            case 4:  return (const void*)warp_row_kernel<DT, NEG, 4, 4, 1>;
            case 8:  return (const void*)warp_row_kernel<DT, NEG, 8, 4, 1>;
            case 16: return (const void*)warp_row_kernel<DT, NEG, 16, 4, 1>;
            default: return (const void*)warp_row_kernel<DT, NEG, 32, 4, 1>;
        }
    }
    if (g.vpl == 8) return (const void*)warp_row_kernel<DT, NEG, 32, 8, 1>;
    if constexpr (DT == DT_F32) {
        if (g.vpl == 16) return (const void*)warp_row_kernel<DT, NEG, 32, 16, 1>;
    }
    return nullptr;
}

#define FS_VPT_TABLE(NAME, KERNEL)                                                          \
    template <int DT, bool NEG> const void* NAME(int vpt) {                                 \
        switch (vpt) {                                                                      \
            case 1: return (const void*)KERNEL<DT, NEG, 1>;                                 \
            case 2: return (const void*)KERNEL<DT, NEG, 2>;                                 \
            case 4: return (const void*)KERNEL<DT, NEG, 4>;                                 \
            case 8: return (const void*)KERNEL<DT, NEG, 8>;                                 \
            case 16:                                                                        \
                if constexpr (DT == DT_F32) return (const void*)KERNEL<DT, NEG, 16>;        \
                else return nullptr;                                                        \
        }                                                                                   \
        return nullptr;                                                                     \
    }
FS_VPT_TABLE(block_fn, block_row_kernel)
FS_VPT_TABLE(block_tma_fn, block_row_tma_kernel)
FS_VPT_TABLE(block_shift_fn, block_row_shift_kernel)

template <int DT> const void* router_fn(const WarpGeom& g) {
    if (g.vpl == 1) return (const void*)router_topk_kernel<DT, 1, 1>;
    if (g.vpl == 2) return (const void*)router_topk_kernel<DT, 1, 2>;
    if (g.vpl == 4) {
        switch (g.lanes) {
            case 1:  return (const void*)router_topk_kernel<DT, 1, 4>;
            case 2:  return (const void*)router_topk_kernel<DT, 2, 4>;
            case 4:  return (const void*)router_topk_kernel<DT, 4, 4>;
            case 8:  return (const void*)router_topk_kernel<DT, 8, 4>;
            case 16: return (const void*)router_topk_kernel<DT, 16, 4>;
            default: return (const void*)router_topk_kernel<DT, 32, 4>;
        }
    }
    if constexpr (DT == DT_F32) {
        if (g.vpl == 8) return (const void*)router_topk_kernel<DT, 32, 8>;
    }
    return nullptr;
}

// k <= 8: the sorting-network kernel, same geometries; FULL when the row fills them exactly
template <int DT, bool FULL> const void* router8_fn(const WarpGeom& g) {
    if (g.vpl == 1) return (const void*)router_top8_kernel<DT, 1, 1, FULL>;
    if (g.vpl == 2) return (const void*)router_top8_kernel<DT, 1, 2, FULL>;
    if (g.vpl == 4) {
        switch (g.lanes) {
            case 1:  return (const void*)router_top8_kernel<DT, 1, 4, FULL>;
            case 2:  return (const void*)router_top8_kernel<DT, 2, 4, FULL>;
            case 4:  return (const void*)router_top8_kernel<DT, 4, 4, FULL>;
            case 8:  return (const void*)router_top8_kernel<DT, 8, 4, FULL>;
            case 16: return (const void*)router_top8_kernel<DT, 16, 4, FULL>;
            default: return (const void*)router_top8_kernel<DT, 32, 4, FULL>;
        }
    }
    if constexpr (DT == DT_F32) {
        if (g.vpl == 8) return (const void*)router_top8_kernel<DT, 32, 8, FULL>;
    }
    return nullptr;
}
template <int DT> const void* router8_fn(const WarpGeom& g, bool full) {
    return full ? router8_fn<DT, true>(g) : router8_fn<DT, false>(g);
}

// Calls f(std::integral_constant<int, DT>, std::bool_constant<NEG>) for the run-time dtype and sign.
template <typename F> const void* by_variant(int dtype, bool neg, F f) {
    auto with_dt = [&](auto dt) -> const void* {
        return neg ? f(dt, std::true_type{}) : f(dt, std::false_type{});
    };
    switch (dtype) {
        case FS_DTYPE_FP32: return with_dt(std::integral_constant<int, DT_F32>{});
        case FS_DTYPE_BF16: return with_dt(std::integral_constant<int, DT_BF16>{});
        default:            return with_dt(std::integral_constant<int, DT_F16>{});
    }
}

// The split-row kernel: whether every block's slice is a whole number of chunks, the kernel
// variant for it, and its dynamic shared memory (slice, chunk mbarriers, per-thread chunk references).
bool smem_row_full(const SmemGeom& g, int dtype, int64_t nvec) {
    const int64_t chunk = int64_t(smem_row_u(dtype)) * g.threads;
    return nvec == int64_t(g.slice) * g.cs && g.slice % chunk == 0;
}
int smem_row_nchunk(const SmemGeom& g, int dtype) {
    const int64_t chunk = int64_t(smem_row_u(dtype)) * g.threads;
    return static_cast<int>((g.slice + chunk - 1) / chunk);
}
const void* smem_row_fn(int dtype, bool neg, const SmemGeom& g, int64_t nvec) {
    const bool full = smem_row_full(g, dtype, nvec);
    return by_variant(dtype, neg, [&](auto dt, auto ng) -> const void* {
        constexpr int DT = decltype(dt)::value;
        constexpr bool NG = decltype(ng)::value;
        return full ? (const void*)smem_row_kernel<DT, NG, true, false> : (const void*)smem_row_kernel<DT, NG, false, false>;
    });
}
// slice rounded up to whole chunks | (warp, chunk) mbarriers | per-thread chunk references
size_t smem_row_stage_bytes(const SmemGeom& g, int dtype) {
    return static_cast<size_t>(smem_row_nchunk(g, dtype)) * smem_row_u(dtype) * g.threads * 16;
}
size_t smem_row_bytes(const SmemGeom& g, int dtype) {
    return smem_row_stage_bytes(g, dtype) + smem_row_tail_bytes(g.threads, smem_row_nchunk(g, dtype));
}

// FS_FORCE_KERNEL (read once): a kernel name or number that replaces the dispatcher's choice.
int forced_kernel() {
    static const int v = [] {
        const char* e = std::getenv("FS_FORCE_KERNEL");
        if (!e || !e[0]) return int(FS_KERNEL_AUTO);
        static const char* names[] = {"auto", "warp", "block", "block_tma", "cluster", "generic"};
        for (int k = 0; k <= FS_KERNEL_GENERIC; ++k)
            if (std::strcmp(e, names[k]) == 0) return k;
        const int k = std::atoi(e);
        return k >= FS_KERNEL_AUTO && k <= FS_KERNEL_GENERIC ? k : int(FS_KERNEL_AUTO);
    }();
    return v;
}

// Rows longer than a cluster's shared memory: segments over a grid that fills the GPU, the
// (reference, sum) pairs of the segments exchanged through the per-device scratch buffer.
struct SplitPlan { LsmParams p; int64_t nseg, seg_vecs; };
bool softmax_split_plan(int sm_count, int* status, const void* x, void* y, int64_t rows, int64_t cols, int dtype, float scale,
                        SplitPlan* out) {
    LsmParams p{};
    p.x = x; p.y = y; p.rows = rows; p.cols = cols;
    p.nvec = cols * elem_size(dtype) / 16;
    p.scale = std::fabs(scale);
    p.c = static_cast<float>(static_cast<double>(p.scale) * kLog2e);
    p.flip = std::signbit(scale) && scale != 0.0f ? (dtype == FS_DTYPE_FP32 ? 0x80000000u : 0x80008000u) : 0u;
    p.status = status; p.pf_rows = 0;
    const int t = kSplitThreads;
    const int64_t target = int64_t(sm_count) * 8;
    int64_t nseg = std::max<int64_t>(1, std::min<int64_t>(1024, (target + rows - 1) / rows));
    const int64_t seg_vecs = ((p.nvec + nseg - 1) / nseg + 4 * t - 1) / (4 * t) * (4 * t);
    nseg = (p.nvec + seg_vecs - 1) / seg_vecs;
    if (rows * nseg > 0x7fffffff || seg_vecs > 0x7fffffff) return false;
    out->p = p; out->nseg = nseg; out->seg_vecs = seg_vecs;
    return true;
}

// The two launches; `part` holds rows * nseg (reference, sum) pairs, every one written by the first
// kernel before the second reads it.
int softmax_split_launch(const SplitPlan& sp, int dtype, float2* part, cudaStream_t st) {
    const void* f1 = nullptr;
    const void* f2 = nullptr;
    switch (dtype) {
        case FS_DTYPE_FP32: f1 = (const void*)sm_partial_kernel<DT_F32>; f2 = (const void*)sm_apply_kernel<DT_F32>; break;
        case FS_DTYPE_BF16: f1 = (const void*)sm_partial_kernel<DT_BF16>; f2 = (const void*)sm_apply_kernel<DT_BF16>; break;
        default:            f1 = (const void*)sm_partial_kernel<DT_F16>; f2 = (const void*)sm_apply_kernel<DT_F16>; break;
    }
    const float2* cpart = part;
    FS_LOGF("softmax %lld x %lld dtype %d: two kernels over %lld segments of %lld vectors per row", (long long)sp.p.rows,
            (long long)sp.p.cols, dtype, (long long)sp.nseg, (long long)sp.seg_vecs);
    int rc = launch(f1, sp.p.rows * sp.nseg, kSplitThreads, 0, 0, st, sp.p, part, static_cast<int>(sp.nseg), static_cast<int>(sp.seg_vecs));
    if (rc == FS_OK)
        rc = launch(f2, sp.p.rows * sp.nseg, kSplitThreads, 0, 0, st, sp.p, cpart, static_cast<int>(sp.nseg), static_cast<int>(sp.seg_vecs));
    return rc;
}

int run_softmax_split(Device& dev, const void* x, void* y, int64_t rows, int64_t cols, int dtype, float scale, cudaStream_t st) {
    SplitPlan sp;
    if (!softmax_split_plan(dev.sm_count, dev.status, x, y, rows, cols, dtype, scale, &sp)) return FS_ERR_UNSUPPORTED;
    std::lock_guard<std::mutex> lk(g_scratch_mu);
    void* buf = nullptr;
    bool capturing = false;
    int rc = scratch_acquire(dev, static_cast<size_t>(rows * sp.nseg) * sizeof(float2), st, &buf, &capturing);
    if (rc != FS_OK) return rc;
    rc = softmax_split_launch(sp, dtype, static_cast<float2*>(buf), st);
    const int rd = scratch_done(dev, st, capturing);
    return rc != FS_OK ? rc : rd;
}

int run(const void* x, void* y, int64_t rows, int64_t cols, int dtype, float scale, cudaStream_t st,
        int kernel, int threads, int cluster, uint32_t dbg_extra_tx = 0u) {
    Device* devp = nullptr;
    int rc = get_device(&devp);
    if (rc != FS_OK) return rc;
    Device& dev = *devp;

    const int esz = elem_size(dtype);
    const bool fast = fast_path_ok(cols, dtype, ptr_align(x), ptr_align(y));
    // The dispatcher's own choice may be downgraded when the device cannot run it (no cluster launch,
    // too little shared memory); a kernel forced by the caller or by FS_FORCE_KERNEL never is.
    bool was_auto = kernel == FS_KERNEL_AUTO;
    if (was_auto) {
        const int forced = forced_kernel();
        if (forced != FS_KERNEL_AUTO) { kernel = forced; was_auto = false; }
        else kernel = select_kernel(cols, dtype, ptr_align(x), ptr_align(y));
    }
    if (kernel != FS_KERNEL_GENERIC && !fast) return FS_ERR_UNSUPPORTED;
    if (threads < 0 || threads % 32 || threads > 1024) return FS_ERR_INVALID_ARG;

    Params p{};
    p.x = x; p.y = y; p.rows = rows; p.cols = cols;
    p.nvec = fast ? cols * esz / 16 : 0;
    p.c = static_cast<float>(static_cast<double>(scale) * kLog2e);
    p.neg = p.c < 0.0f ? 1 : 0;
    p.status = dev.status;
    p.q_offset = 0;
    p.pf_rows = 0;
    p.dbg_extra_tx = dbg_extra_tx;
    p.early_pf = early_prefetch_enabled();
    p.wait_polls = dev.wait_polls.load(std::memory_order_relaxed);
    const int64_t max_grid = 0x7fffffff;

    // One block per row with element-wise accesses; vector-aligned rows of 1 MiB or more that no
    // cluster holds (the dispatcher's own choice only) are cut into segments over two kernels instead.
    const auto run_generic = [&](bool allow_split, int t) -> int {
        if (allow_split && fast && cols * esz >= (int64_t(1) << 20)) return run_softmax_split(dev, x, y, rows, cols, dtype, scale, st);
        // Rows whose byte length is not a multiple of 16, in tensors that are themselves 16-byte aligned: the block
        // kernel on the aligned vectors that cover each row (block_row_shift_kernel), as long as a block's registers
        // hold the row. A zero scale, a forced block size and FS_SHIFT=0 keep the element-wise kernel.
        if (t == 0 && shift_enabled() && (cols * esz) % 16 != 0 && cols * esz <= kSpanMaxRowBytes && ptr_align(x) >= 16 &&
            ptr_align(y) >= 16) {
            // short rows: a block takes 128 consecutive rows as one span of the tensor (span_rows_kernel)
            const void* fn = by_variant(dtype, p.neg, [&](auto dt, auto ng) -> const void* {
                return (const void*)span_rows_kernel<decltype(dt)::value, decltype(ng)::value>; });
            const int tb = 128;        // (32 or 64 rows per block change nothing: the per-thread loops are what takes the time)
            const size_t smem = (size_t(tb) * size_t(cols * esz) + 15 + 15) / 16 * 16 + 16;
            const int64_t grid = (rows + tb - 1) / tb;
            if (grid <= max_grid && smem <= static_cast<size_t>(dev.smem_optin) - 2048) {
                int bps = 0;
                if ((rc = blocks_per_sm(dev, fn, tb, smem, &bps)) != FS_OK) return rc;
                FS_LOGF("softmax %lld x %lld dtype %d: spans of %d short rows (rows not a multiple of 16 bytes), %zu B shared",
                        (long long)rows, (long long)cols, dtype, tb, smem);
                return launch(fn, grid, tb, smem, 0, st, p, int64_t(rows * cols * esz / 16));
            }
        }
        const bool shift_ok = t == 0 && shift_enabled() && p.c != 0.0f && (cols * esz) % 16 != 0 && ptr_align(x) >= 16 &&
                              ptr_align(y) >= 16 && cols < (int64_t(1) << 24);
        const int64_t nvr_max = (cols + 2 * (16 / esz - 1)) / (16 / esz);      // vectors that cover a row, at most
        if (shift_ok && dev.cluster_ok && cols * esz > shift_block_max_row_bytes()) {
            // long rows: the split-row kernel on the aligned vectors that cover each row (one cluster per row)
            SmemGeom sg;
            if (smem_geom(nvr_max, dtype, 0, 0, &sg) && rows <= max_grid / sg.cs) {
                const void* fn = by_variant(dtype, p.neg, [&](auto dt, auto ng) -> const void* {
                    return (const void*)smem_row_kernel<decltype(dt)::value, decltype(ng)::value, false, false, true>; });
                const size_t stage_bytes = smem_row_stage_bytes(sg, dtype);
                const size_t smem = smem_row_bytes(sg, dtype);
                if (smem <= static_cast<size_t>(dev.smem_optin) - 2048) {
                    int ncl = 0;
                    if ((rc = active_clusters(dev, fn, sg.threads, smem, sg.cs, &ncl)) != FS_OK) return rc;
                    Params ps = p;
                    ps.nvec = 0;                                   // the kernel takes every row's own vector range
                    ps.tensor_vecs = rows * cols * esz / 16;
                    ps.pf_rows = prefetch_rows(ncl);
                    set_first_wave_lag(ps, ncl, nvr_max * 16);
                    FS_LOGF("softmax %lld x %lld dtype %d: split-row kernel on shifted vectors (rows not a multiple of 16 bytes), %d blocks per row x %d "
                            "threads, %zu B shared", (long long)rows, (long long)cols, dtype, sg.cs, sg.threads, smem);
                    return launch(fn, rows * sg.cs, sg.threads, smem, sg.cs, st, ps, static_cast<uint32_t>(stage_bytes), sg.slice,
                                  smem_row_nchunk(sg, dtype));
                }
            }
        }
        if (shift_ok) {
            BlockGeom g;
            if (block_geom(nvr_max + 1, dtype, 0, &g)) {
                const void* fn = by_variant(dtype, p.neg, [&](auto dt, auto ng) { return block_shift_fn<decltype(dt)::value, decltype(ng)::value>(g.vpt); });
                if (fn) {
                    FS_LOGF("softmax %lld x %lld dtype %d: block kernel on shifted vectors (rows not a multiple of 16 bytes), %d threads x %d vectors",
                            (long long)rows, (long long)cols, dtype, g.threads, g.vpt);
                    return launch(fn, std::min<int64_t>(rows, max_grid), g.threads, 0, 0, st, p, int64_t(rows * cols * esz / 16));
                }
            }
        }
        const void* fn = by_variant(dtype, p.neg, [&](auto dt, auto ng) { return (const void*)generic_row_kernel<decltype(dt)::value, decltype(ng)::value, false>; });
        if (t == 0) {
            t = 32;
            while (t < 1024 && cols > int64_t(t) * 8) t <<= 1;
        }
        FS_LOGF("softmax %lld x %lld dtype %d: generic kernel, %d threads per row", (long long)rows, (long long)cols, dtype, t);
        return launch(fn, std::min<int64_t>(rows, max_grid), t, 0, 0, st, p);
    };

    switch (kernel) {
        case FS_KERNEL_WARP: {
            WarpGeom g;
            if (!warp_geom(p.nvec, dtype, &g)) return FS_ERR_UNSUPPORTED;
            const void* fn = by_variant(dtype, p.neg, [&](auto dt, auto ng) { return warp_fn<decltype(dt)::value, decltype(ng)::value>(g); });
            if (!fn) return FS_ERR_UNSUPPORTED;
            const int t = threads ? threads : 128;
            if (t > 256) return FS_ERR_UNSUPPORTED;
            const int64_t rows_per_tile = int64_t(32 / g.lanes) * g.r;
            const int64_t tiles = (rows + rows_per_tile - 1) / rows_per_tile;
            const int64_t grid = std::min<int64_t>((tiles + (t / 32) - 1) / (t / 32), max_grid);
            FS_LOGF("softmax %lld x %lld dtype %d: warp kernel, %d lanes x %d vectors per row, %d rows per group, grid %lld x %d",
                    (long long)rows, (long long)cols, dtype, g.lanes, g.vpl, g.r, (long long)grid, t);
            return launch(fn, grid, t, 0, 0, st, p);
        }
        case FS_KERNEL_BLOCK: {
            BlockGeom g;
            if (!block_geom(p.nvec, dtype, threads, &g)) return FS_ERR_UNSUPPORTED;
            const void* fn = by_variant(dtype, p.neg, [&](auto dt, auto ng) { return block_fn<decltype(dt)::value, decltype(ng)::value>(g.vpt); });
            if (!fn) return FS_ERR_UNSUPPORTED;
            const int64_t grid = std::min<int64_t>(rows, max_grid);
            int bps = 0;
            if ((rc = blocks_per_sm(dev, fn, g.threads, 0, &bps)) != FS_OK) return rc;
            p.pf_rows = prefetch_rows(dev.sm_count * bps);
            FS_LOGF("softmax %lld x %lld dtype %d: block kernel, %d threads x %d vectors, %d blocks per SM", (long long)rows,
                    (long long)cols, dtype, g.threads, g.vpt, bps);
            return launch(fn, grid, g.threads, 0, 0, st, p);
        }
        case FS_KERNEL_BLOCK_TMA: {
            const size_t smem_cap = static_cast<size_t>(dev.smem_optin) - 2048;   // room for the static part
            if (was_auto && softmax_tile_wanted(dtype, p.nvec)) {
                // the dispatcher's own choice for 16-bit rows of 4-12 KiB: four rows per block in shared memory,
                // each brought by its own bulk copy and worked on by one warp
                const void* fn = by_variant(dtype, p.neg, [&](auto dt, auto ng) -> const void* {
                    constexpr int DT = decltype(dt)::value;
                    if constexpr (DT == DT_F32) return nullptr;
                    else return (const void*)softmax_tile_kernel<DT, decltype(ng)::value>; });
                const int t = 128;
                const size_t smem = size_t(t / 32) * size_t(p.nvec) * 16 + size_t(t / 32) * 8;
                const int64_t grid = (rows + (t / 32) - 1) / (t / 32);
                if (fn && smem <= smem_cap && grid <= max_grid) {
                    int bps = 0;
                    if ((rc = blocks_per_sm(dev, fn, t, smem, &bps)) != FS_OK) return rc;
                    p.pf_rows = prefetch_rows(dev.sm_count * bps) * (t / 32);
                    set_first_wave_lag(p, dev.sm_count * bps, (t / 32) * p.nvec * 16);
                    FS_LOGF("softmax %lld x %lld dtype %d: four rows per block from shared memory, a warp per row, %d blocks per SM",
                            (long long)rows, (long long)cols, dtype, bps);
                    return launch(fn, grid, t, smem, 0, st, p);
                }
                // (too little shared memory on this device: the block-per-row form below takes the row)
            }
            BlockGeom g;
            if (!block_geom(p.nvec, dtype, threads, &g)) return FS_ERR_UNSUPPORTED;
            const void* fn = by_variant(dtype, p.neg, [&](auto dt, auto ng) { return block_tma_fn<decltype(dt)::value, decltype(ng)::value>(g.vpt); });
            if (!fn) return FS_ERR_UNSUPPORTED;
            const size_t stage_bytes = static_cast<size_t>(p.nvec) * 16;
            if (stage_bytes > (size_t(1) << 20) - 16) return FS_ERR_UNSUPPORTED;
            const int nstage = 1;                   // one row per block: a single stage
            if (stage_bytes + 8 > smem_cap) {
                if (!was_auto) return FS_ERR_UNSUPPORTED;
                FS_LOGF("softmax: a %zu B row exceeds the device's shared memory per block: generic path", stage_bytes);
                return run_generic(false, 0);
            }
            const size_t smem = nstage * stage_bytes + size_t(nstage) * 8;
            int bps = 0;
            if ((rc = blocks_per_sm(dev, fn, g.threads, smem, &bps)) != FS_OK) return rc;
            const int64_t grid = std::min<int64_t>(rows, max_grid);
            set_first_wave_lag(p, dev.sm_count * bps, p.nvec * 16);
            FS_LOGF("softmax %lld x %lld dtype %d: block kernel fed by bulk copies, %d threads x %d vectors, %d blocks per SM",
                    (long long)rows, (long long)cols, dtype, g.threads, g.vpt, bps);
            return launch(fn, grid, g.threads, smem, 0, st, p, nstage, static_cast<uint32_t>(stage_bytes));
        }
        case FS_KERNEL_CLUSTER: {
            // A device without cluster launch still runs the one-block form (cluster size 1) on rows
            // that fit one block's shared memory; the dispatcher sends everything else to the generic
            // kernels then, and does the same when the device's shared memory is too small.
            if (!dev.cluster_ok) {
                if (cluster > 1 || (!was_auto && cluster == 0)) return FS_ERR_UNSUPPORTED;
                cluster = 1;
            }
            SmemGeom sg;
            if (smem_geom(p.nvec, dtype, threads, cluster, &sg)) {
                // a slice that is not a whole number of chunks is padded with -inf, which a zero
                // scale would turn into NaN: that one case goes to the generic kernel
                const bool zero_scale_ragged = p.c == 0.0f && !smem_row_full(sg, dtype, p.nvec);
                if (zero_scale_ragged && !was_auto) return FS_ERR_UNSUPPORTED;
                if (!zero_scale_ragged) {
                    const void* fn = smem_row_fn(dtype, p.neg, sg, p.nvec);
                    const size_t stage_bytes = smem_row_stage_bytes(sg, dtype);
                    const size_t smem = smem_row_bytes(sg, dtype);
                    if (smem > static_cast<size_t>(dev.smem_optin) - 2048) {
                        if (!was_auto) return FS_ERR_UNSUPPORTED;
                        FS_LOGF("softmax: %zu B of shared memory per block exceed the device's limit: generic path", smem);
                        return run_generic(true, 0);
                    }
                    int ncl = 0;
                    if (dev.cluster_ok) {
                        if ((rc = active_clusters(dev, fn, sg.threads, smem, sg.cs, &ncl)) != FS_OK) return rc;
                    } else {                       // plain launch of the one-block form
                        if ((rc = blocks_per_sm(dev, fn, sg.threads, smem, &ncl)) != FS_OK) return rc;
                        ncl *= dev.sm_count;
                    }
                    const int64_t clusters = std::min<int64_t>(rows, max_grid / sg.cs);
                    p.pf_rows = prefetch_rows(ncl);
                    set_first_wave_lag(p, ncl, p.nvec * 16);
                    FS_LOGF("softmax %lld x %lld dtype %d: split-row kernel, %d blocks per row x %d threads, slice %d B, %zu B shared, "
                            "%d resident clusters", (long long)rows, (long long)cols, dtype, sg.cs, sg.threads, sg.slice * 16, smem, ncl);
                    return launch(fn, clusters * sg.cs, sg.threads, smem, dev.cluster_ok ? sg.cs : 0, st, p,
                                  static_cast<uint32_t>(stage_bytes), sg.slice, smem_row_nchunk(sg, dtype));
                }
                return run_generic(false, 0);
            }
            if (!dev.cluster_ok) {
                if (!was_auto) return FS_ERR_UNSUPPORTED;
                FS_LOGF("softmax: no cluster launch on this device and the row does not fit one block: generic path");
                return run_generic(true, 0);
            }
            return FS_ERR_UNSUPPORTED;           // no geometry holds this row in a cluster's shared memory
        }
        case FS_KERNEL_GENERIC:
            return run_generic(was_auto, threads);
        default:
            return FS_ERR_INVALID_ARG;
    }
}

// Causal softmax: the split-row kernel (one cluster per row) when the tensors are vector-aligned
// and the row fits its shared memory, the generic kernel otherwise.
int run_causal(const void* x, void* y, int64_t rows, int64_t cols, int64_t q_offset, int dtype, float scale,
               cudaStream_t st) {
    Device* devp = nullptr;
    int rc = get_device(&devp);
    if (rc != FS_OK) return rc;
    Device& dev = *devp;
    const int esz = elem_size(dtype);
    const bool fast = fast_path_ok(cols, dtype, ptr_align(x), ptr_align(y));
    Params p{};
    p.x = x; p.y = y; p.rows = rows; p.cols = cols;
    p.nvec = fast ? cols * esz / 16 : 0;
    p.c = static_cast<float>(static_cast<double>(scale) * kLog2e);
    p.neg = p.c < 0.0f ? 1 : 0;
    p.status = dev.status;
    p.q_offset = q_offset;
    p.pf_rows = 0;
    p.wait_polls = kDefaultWaitPolls;
    p.early_pf = early_prefetch_enabled();
    SmemGeom sg;
    // (a zero scale goes to the generic kernel: the split kernel masks with -inf, and 0 * -inf is NaN)
    if (fast && p.c != 0.0f && dev.cluster_ok && smem_geom(p.nvec, dtype, 0, 0, &sg) && rows <= 0x7fffffff / sg.cs) {
        const void* fn = by_variant(dtype, p.neg, [&](auto dt, auto ng) -> const void* {
            return (const void*)smem_row_kernel<decltype(dt)::value, decltype(ng)::value, false, true>; });
        const size_t smem = smem_row_bytes(sg, dtype);
        if (smem <= static_cast<size_t>(dev.smem_optin) - 2048) {
            int ncl = 0;
            if ((rc = active_clusters(dev, fn, sg.threads, smem, sg.cs, &ncl)) != FS_OK) return rc;
            p.pf_rows = prefetch_rows(ncl);
            return launch(fn, rows * sg.cs, sg.threads, smem, sg.cs, st, p,
                          static_cast<uint32_t>(smem_row_stage_bytes(sg, dtype)), sg.slice, smem_row_nchunk(sg, dtype));
        }
    }
    const void* fn = by_variant(dtype, p.neg, [&](auto dt, auto ng) -> const void* {
        return (const void*)generic_row_kernel<decltype(dt)::value, decltype(ng)::value, true>; });
    int t = 32;
    while (t < 1024 && cols > int64_t(t) * 8) t <<= 1;
    return launch(fn, std::min<int64_t>(rows, 0x7fffffff), t, 0, 0, st, p);
}

int validate(const void* x, const void* y, int64_t rows, int64_t cols, int dtype, float scale) {
    if (rows < 0 || cols < 0) return FS_ERR_INVALID_ARG;
    if (dtype != FS_DTYPE_FP32 && dtype != FS_DTYPE_BF16 && dtype != FS_DTYPE_FP16) return FS_ERR_INVALID_ARG;
    if (!std::isfinite(scale)) return FS_ERR_INVALID_ARG;
    if (rows == 0 || cols == 0) return FS_OK;
    if (!x || !y) return FS_ERR_INVALID_ARG;
    if (cols > (int64_t(1) << 40) || rows > (int64_t(1) << 40)) return FS_ERR_INVALID_ARG;
    const unsigned __int128 total = (unsigned __int128)rows * (unsigned __int128)cols * elem_size(dtype);
    if (total > (unsigned __int128)1 << 62) return FS_ERR_INVALID_ARG;
    const uintptr_t a = reinterpret_cast<uintptr_t>(x), b = reinterpret_cast<uintptr_t>(y);
    const uintptr_t n = static_cast<uintptr_t>(total);
    if (a != b && a < b + n && b < a + n) return FS_ERR_INVALID_ARG;   // partial overlap
    return FS_OK;
}

// FS_CHECK=1: every tensor pointer must be memory the current device can address (device or managed
// memory of this device, or mapped pinned host memory). One driver query per pointer: slow, off by default.
int check_ptrs(std::initializer_list<const void*> ptrs) {
    if (!check_enabled()) return FS_OK;
    int d = 0;
    FS_CUDA(cudaGetDevice(&d));
    for (const void* q : ptrs) {
        if (!q) continue;
        cudaPointerAttributes a{};
        FS_CUDA(cudaPointerGetAttributes(&a, q));
        const bool ok = (a.type == cudaMemoryTypeDevice && a.device == d) || a.type == cudaMemoryTypeManaged ||
                        (a.type == cudaMemoryTypeHost && a.devicePointer != nullptr);
        if (!ok) {
            FS_LOGF("FS_CHECK: %p is not addressable by device %d (memory type %d, device %d)", q, d, int(a.type), a.device);
            return FS_ERR_INVALID_ARG;
        }
    }
    return FS_OK;
}
#define FS_CHECK_PTRS(...) do { const int c__ = check_ptrs({__VA_ARGS__}); if (c__ != FS_OK) return c__; } while (0)

}  // namespace

// ---------------------------------------------------------------------------------------------
// fs_softmax_static: scratch in a fixed device array instead of allocated memory
// ---------------------------------------------------------------------------------------------
// Two things the other entry points keep in memory from cudaMalloc live in the array below, which is
// part of the loaded module (FS_STATIC_SCRATCH_BYTES on every GPU that loads the library, held until
// the process exits): the status word of the bounded waits (word 0), and, from byte 256 on, the
// (reference, sum) pairs that the two kernels of the long-row path hand to each other. In host code the array's name is only a handle for the runtime, not a device
// address: the address a kernel can use comes from cudaGetSymbolAddress, asked once per device with
// that device current.
constexpr int kStaticScratchWords = FS_STATIC_SCRATCH_BYTES / 4;
constexpr int kStaticPairOffsetWords = 64;                       // pairs start 256 bytes in
static_assert((kStaticScratchWords - kStaticPairOffsetWords) / 2 == FS_STATIC_MAX_PAIRS, "header and array disagree");
static __device__ __align__(256) int fs_static_scratch[kStaticScratchWords];

namespace {

struct StaticDevice {
    bool ready = false;
    int sm_count = 0;
    int smem_optin = 0;
    int cluster_ok = 0;
    int* scratch = nullptr;              // device address of fs_static_scratch on this device
    bool configured[3][2][2] = {};       // split-row kernel variants whose attributes are set
    // resident clusters per launch geometry (an occupancy query, no allocation), for the prefetch distance and the lag
    struct Geo { const void* fn; int threads, cs; size_t smem; int ncl; } geo[16] = {};
    int ngeo = 0;
};
StaticDevice g_static[kMaxDevices];
std::mutex g_static_mu;

// First use on a device: queries and the symbol's address, no allocation.
int get_static_device(StaticDevice** out) {
    int d = 0;
    FS_CUDA(cudaGetDevice(&d));
    if (d < 0 || d >= kMaxDevices) return FS_ERR_UNSUPPORTED;
    StaticDevice& sd = g_static[d];
    if (!sd.ready) {
        FS_CUDA(cudaDeviceGetAttribute(&sd.sm_count, cudaDevAttrMultiProcessorCount, d));
        FS_CUDA(cudaDeviceGetAttribute(&sd.smem_optin, cudaDevAttrMaxSharedMemoryPerBlockOptin, d));
        FS_CUDA(cudaDeviceGetAttribute(&sd.cluster_ok, cudaDevAttrClusterLaunch, d));
        void* addr = nullptr;
        FS_CUDA(cudaGetSymbolAddress(&addr, fs_static_scratch));
        sd.scratch = static_cast<int*>(addr);
        sd.ready = true;
    }
    *out = &sd;
    return FS_OK;
}

}  // namespace

// =============================================================================================
// C ABI
// =============================================================================================

// ---------------------------------------------------------------------------------------------
// row normalisations
// ---------------------------------------------------------------------------------------------
namespace {

// Warp-per-row geometry of the normalisation kernels: sub-warp groups with up to four vectors per
// lane for short rows, whole warps with up to eight (any count, so that no lane idles on rows of
// 96, 160 or 192 vectors) up to 4 KiB.
bool norm_warp_geom(int64_t nvec, int dtype, WarpGeom* g) {
    if (nvec < 1 || nvec > 256) return false;
    if (nvec <= 64) return warp_geom(nvec, dtype, g) && g->vpl <= 4;
    g->lanes = 32; g->vpl = static_cast<int>((nvec + 31) / 32); g->r = 1;
    return true;
}

template <int DT, int AFF> const void* norm_warp_fn(const WarpGeom& g) {
    if (g.lanes == 32) {
        switch (g.vpl) {
            case 1: return (const void*)norm_warp_kernel<DT, 32, 1, AFF>;
            case 2: return (const void*)norm_warp_kernel<DT, 32, 2, AFF>;
            case 3: return (const void*)norm_warp_kernel<DT, 32, 3, AFF>;
            case 4: return (const void*)norm_warp_kernel<DT, 32, 4, AFF>;
            case 5: return (const void*)norm_warp_kernel<DT, 32, 5, AFF>;
            case 6: return (const void*)norm_warp_kernel<DT, 32, 6, AFF>;
            case 7: return (const void*)norm_warp_kernel<DT, 32, 7, AFF>;
            case 8: return (const void*)norm_warp_kernel<DT, 32, 8, AFF>;
            default: return nullptr;
        }
    }
    if (g.vpl == 1) return (const void*)norm_warp_kernel<DT, 1, 1, AFF>;
    if (g.vpl == 2) return (const void*)norm_warp_kernel<DT, 1, 2, AFF>;
    if (g.vpl != 4) return nullptr;
    switch (g.lanes) {
        case 1:  return (const void*)norm_warp_kernel<DT, 1, 4, AFF>;
        case 2:  return (const void*)norm_warp_kernel<DT, 2, 4, AFF>;
        case 4:  return (const void*)norm_warp_kernel<DT, 4, 4, AFF>;
        case 8:  return (const void*)norm_warp_kernel<DT, 8, 4, AFF>;
        default: return (const void*)norm_warp_kernel<DT, 16, 4, AFF>;
    }
}

template <int DT> const void* norm_smem_fn(bool full, int aff) {
    if (full) {
        return aff == 0 ? (const void*)norm_smem_kernel<DT, true, 0> : aff == 1 ? (const void*)norm_smem_kernel<DT, true, 1>
                                                                                : (const void*)norm_smem_kernel<DT, true, 2>;
    }
    return aff == 0 ? (const void*)norm_smem_kernel<DT, false, 0> : aff == 1 ? (const void*)norm_smem_kernel<DT, false, 1>
                                                                            : (const void*)norm_smem_kernel<DT, false, 2>;
}

template <int DT> const void* norm_apply_fn(int aff) {
    return aff == 0 ? (const void*)norm_apply_kernel<DT, 0> : aff == 1 ? (const void*)norm_apply_kernel<DT, 1>
                                                                        : (const void*)norm_apply_kernel<DT, 2>;
}

// Rows the warp-per-row-from-shared-memory kernel takes (16-byte vectors per row): 4-11 KiB.
// Measured on B200 (256 MiB per direction, gamma and beta present, copy = 80 us), against the
// kernels on either side of the range: bf16 rows of 4 / 5 / 6 / 8 / 10 KiB 83 / 84 / 81 / 82 / 83 us
// (register-resident warp kernels: 93 / 92 / 90 / 100 / 105), fp32 rows of 6 / 8 / 10 KiB 82 / 83 / 83
// (split-row kernel: 118 / 98 / 90); from 12 KiB on the split-row kernel is level or ahead, below
// 4 KiB four rows per block are too few bytes in flight (3 KiB bf16 rows: 97 against 90).
// FS_NORM_TILE "lo:hi" (read once) overrides the range (lo < vectors <= hi), "0" turns the kernel off.
bool norm_tile_wanted(int dtype, int64_t nvec) {
    static const std::pair<int64_t, int64_t> ov = [] {
        const char* e = std::getenv("FS_NORM_TILE");
        if (!e) return std::pair<int64_t, int64_t>(-1, -1);
        long lo = 0, hi = 0;
        if (std::sscanf(e, "%ld:%ld", &lo, &hi) == 2) return std::pair<int64_t, int64_t>(lo, hi);
        return std::pair<int64_t, int64_t>(0, 0);
    }();
    if (ov.first >= 0) return nvec > ov.first && nvec <= ov.second;
    (void)dtype;
    return nvec >= 256 && nvec <= 704;
}

// The same for fs_softmax_masked: 16-bit rows of 4-10 KiB. Measured (256 MiB per direction, copy =
// 80 us; mask of 64 rows shared by all others): bf16 rows of 4 / 5 / 6 / 8 / 10 KiB 94 / 96 / 91 / 98 / 103 us
// against 96 / 108 / 116 / 130 / 112 with the row packed in registers; from 11 KiB on and for fp32 rows
// (82-98 against 81-93) the other kernels are level or ahead.
// FS_MASKED_TILE "lo:hi" overrides the range, "0" turns the kernel off.
bool masked_tile_wanted(int dtype, int64_t nvec) {
    static const std::pair<int64_t, int64_t> ov = [] {
        const char* e = std::getenv("FS_MASKED_TILE");
        if (!e) return std::pair<int64_t, int64_t>(-1, -1);
        long lo = 0, hi = 0;
        if (std::sscanf(e, "%ld:%ld", &lo, &hi) == 2) return std::pair<int64_t, int64_t>(lo, hi);
        return std::pair<int64_t, int64_t>(0, 0);
    }();
    if (ov.first >= 0) return nvec > ov.first && nvec <= ov.second;
    return dtype != FS_DTYPE_FP32 && nvec >= 256 && nvec <= 640;
}

// The same for fs_softmax_backward (the dy and the y row of a warp in shared memory): rows of 4-8 KiB.
// Measured (256 MiB per tensor, a copy of the same bytes = 115 us): rows of 5 / 6 / 7 / 8 KiB 118 / 118 / 117 / 117 us
// against 150 / 135 / 126 / 120 on the split-row kernel; level from 10 KiB on. FS_SMB_TILE "lo:hi" overrides.
bool smb_tile_wanted(int64_t nvec) {
    static const std::pair<int64_t, int64_t> ov = [] {
        const char* e = std::getenv("FS_SMB_TILE");
        if (!e) return std::pair<int64_t, int64_t>(-1, -1);
        long lo = 0, hi = 0;
        if (std::sscanf(e, "%ld:%ld", &lo, &hi) == 2) return std::pair<int64_t, int64_t>(lo, hi);
        return std::pair<int64_t, int64_t>(0, 0);
    }();
    if (ov.first >= 0) return nvec > ov.first && nvec <= ov.second;
    return nvec > 256 && nvec <= 512;
}

// The same for fs_log_softmax and fs_softmax_f32out: rows of 4-12 KiB. Measured (256 MiB per direction,
// copy = 80 us): bf16 rows of 5 / 6 / 7 / 8 / 10 / 12 KiB 82 / 82 / 82 / 81 / 82 / 82 us against 88 / 83 / 89 / 86 / 93 / 83
// with the row packed in registers or split over a block; fp32 rows of 8 / 10 KiB 81 / 81 against 83 / 88;
// from 14 KiB on the split-row kernel is ahead (bf16 86 / 79 against 91 / 90). FS_LSM_TILE "lo:hi" overrides.
bool lsm_tile_wanted(int dtype, int64_t nvec) {
    static const std::pair<int64_t, int64_t> ov = [] {
        const char* e = std::getenv("FS_LSM_TILE");
        if (!e) return std::pair<int64_t, int64_t>(-1, -1);
        long lo = 0, hi = 0;
        if (std::sscanf(e, "%ld:%ld", &lo, &hi) == 2) return std::pair<int64_t, int64_t>(lo, hi);
        return std::pair<int64_t, int64_t>(0, 0);
    }();
    if (ov.first >= 0) return nvec > ov.first && nvec <= ov.second;
    (void)dtype;
    return nvec > 256 && nvec <= 768;
}

// FS_NORM_SPLIT=0 / 1 (read once) forces the choice for experiments.
bool norm_split_wanted(const Device& dev, int64_t rows, int64_t nvec, bool smem_ok, int cs) {
    static const int forced = [] { const char* e = std::getenv("FS_NORM_SPLIT"); return e ? std::atoi(e) : -1; }();
    if (forced == 0) return false;
    if (forced == 1) return true;
    // Rows that a cluster's shared memory holds stay there: measured on B200 (one image, 32 groups of
    // 0.5 / 1 / 2 MiB), the cluster kernel takes 12.7 / 21.3 / 43.9 us where the two-kernel form takes
    // 19.4 / 29.5 / 46.4 (two launches, and the second read does not stay in L2).
    (void)dev; (void)rows; (void)cs;
    return !smem_ok && nvec * 16 >= (int64_t(1) << 20);
}

template <typename F> const void* by_dtype(int dtype, F f) {
    switch (dtype) {
        case FS_DTYPE_FP32: return f(std::integral_constant<int, DT_F32>{});
        case FS_DTYPE_BF16: return f(std::integral_constant<int, DT_BF16>{});
        default:            return f(std::integral_constant<int, DT_F16>{});
    }
}

// Rows of `cols` elements; affine parameters per column (aff 1), per run of run_elems elements with
// aff_rows rows per sample (aff 2), or none (aff 0).
int run_norm(const void* x, const void* gamma, const void* beta, void* y, int64_t rows, int64_t cols, int dtype,
             float eps, int aff, int64_t run_elems, int64_t aff_rows, cudaStream_t st) {
    Device* devp = nullptr;
    int rc = get_device(&devp);
    if (rc != FS_OK) return rc;
    Device& dev = *devp;
    const int esz = elem_size(dtype);
    const int ve = 16 / esz;
    bool fast = fast_path_ok(cols, dtype, ptr_align(x), ptr_align(y));
    if (aff == 1) fast = fast && (!gamma || ptr_align(gamma) >= 16) && (!beta || ptr_align(beta) >= 16);
    if (aff == 2) fast = fast && run_elems % ve == 0;
    NormParams p{};
    p.x = x; p.y = y; p.gamma = gamma; p.beta = beta; p.rows = rows; p.cols = cols;
    p.nvec = fast ? cols * esz / 16 : 0;
    p.eps = eps; p.run_elems = run_elems; p.aff_rows = aff_rows;
    p.status = dev.status; p.pf_rows = 0;
    // rows of 4-11 KiB: a warp per row from shared memory, four rows per block
    if (fast && aff != 2 && norm_tile_wanted(dtype, p.nvec)) {
        const void* fn = by_dtype(dtype, [&](auto dt) -> const void* {
            return aff ? (const void*)norm_tile_kernel<decltype(dt)::value, 1> : (const void*)norm_tile_kernel<decltype(dt)::value, 0>; });
        const int t = 128;
        const size_t smem = size_t(t / 32) * size_t(p.nvec) * 16 + size_t(t / 32) * 8;
        int bps = 0;
        if ((rc = blocks_per_sm(dev, fn, t, smem, &bps)) != FS_OK) return rc;
        const int64_t grid = (rows + (t / 32) - 1) / (t / 32);
        if (grid <= 0x7fffffff) {
            p.pf_rows = prefetch_rows(dev.sm_count * bps) * (t / 32);
            set_first_wave_lag(p, dev.sm_count * bps, (t / 32) * p.nvec * 16);
            return launch(fn, grid, t, smem, 0, st, p);
        }
    }
    WarpGeom wg;
    if (fast && aff != 2 && norm_warp_geom(p.nvec, dtype, &wg)) {
        const void* fn = by_dtype(dtype, [&](auto dt) -> const void* {
            return aff ? norm_warp_fn<decltype(dt)::value, 1>(wg) : norm_warp_fn<decltype(dt)::value, 0>(wg); });
        if (fn) {
            const int t = 128;
            const int64_t groups = (rows + (32 / wg.lanes) - 1) / (32 / wg.lanes);
            const int64_t grid = std::min<int64_t>((groups + (t / 32) - 1) / (t / 32), 0x7fffffff);
            return launch(fn, grid, t, 0, 0, st, p);
        }
    }
    SmemGeom sg;
    const bool smem_ok = fast && dev.cluster_ok && smem_geom(p.nvec, dtype, 0, 0, &sg) && rows <= 0x7fffffff / sg.cs;
    // Few, very long rows (group_norm of a large image): a cluster per row leaves most of the GPU
    // idle, or the row does not fit a cluster's shared memory at all. Then the rows are cut into
    // segments over a grid that fills the GPU, with the partial statistics exchanged through the
    // per-device scratch buffer between two kernels.
    if (fast && norm_split_wanted(dev, rows, p.nvec, smem_ok, smem_ok ? sg.cs : 0)) {
        const int t = 256;
        const int64_t target = int64_t(dev.sm_count) * 8;
        int64_t nseg = std::max<int64_t>(1, std::min<int64_t>(1024, (target + rows - 1) / rows));
        int64_t seg_vecs = ((p.nvec + nseg - 1) / nseg + 4 * t - 1) / (4 * t) * (4 * t);
        nseg = (p.nvec + seg_vecs - 1) / seg_vecs;
        if (rows * nseg <= 0x7fffffff) {
            std::lock_guard<std::mutex> lk(g_scratch_mu);
            void* buf = nullptr;
            bool capturing = false;
            if ((rc = scratch_acquire(dev, static_cast<size_t>(rows * nseg) * sizeof(float4), st, &buf, &capturing)) != FS_OK) return rc;
            float4* part = static_cast<float4*>(buf);
            const void* f1 = by_dtype(dtype, [&](auto dt) -> const void* { return (const void*)norm_partial_kernel<decltype(dt)::value>; });
            const void* f2 = by_dtype(dtype, [&](auto dt) -> const void* { return norm_apply_fn<decltype(dt)::value>(aff); });
            const float4* cpart = part;
            rc = launch(f1, rows * nseg, t, 0, 0, st, p, part, static_cast<int>(nseg), static_cast<int>(seg_vecs));
            if (rc == FS_OK) rc = launch(f2, rows * nseg, t, 0, 0, st, p, cpart, static_cast<int>(nseg), static_cast<int>(seg_vecs));
            const int rd = scratch_done(dev, st, capturing);
            return rc != FS_OK ? rc : rd;
        }
    }
    if (smem_ok) {
        const bool full = smem_row_full(sg, dtype, p.nvec);
        const void* fn = by_dtype(dtype, [&](auto dt) -> const void* { return norm_smem_fn<decltype(dt)::value>(full, aff); });
        const size_t stage_bytes = smem_row_stage_bytes(sg, dtype);
        const size_t smem = stage_bytes + size_t(kNormMaxChunks) * 8;
        if (smem <= static_cast<size_t>(dev.smem_optin) - 2048) {
            int ncl = 0;
            if ((rc = active_clusters(dev, fn, sg.threads, smem, sg.cs, &ncl)) != FS_OK) return rc;
            p.pf_rows = prefetch_rows(ncl);
            set_first_wave_lag(p, ncl, p.nvec * 16);
            return launch(fn, rows * sg.cs, sg.threads, smem, sg.cs, st, p, static_cast<uint32_t>(stage_bytes), sg.slice,
                          smem_row_nchunk(sg, dtype));
        }
    }
    const void* fn = by_dtype(dtype, [&](auto dt) -> const void* { return (const void*)norm_generic_kernel<decltype(dt)::value>; });
    int t = 32;
    while (t < 1024 && cols > int64_t(t) * 8) t <<= 1;
    p.nvec = 0;
    return launch(fn, std::min<int64_t>(rows, 0x7fffffff), t, 0, 0, st, p, aff);
}

int validate_norm(const void* x, const void* y, int64_t rows, int64_t cols, int dtype, float eps) {
    if (rows < 0 || cols < 0) return FS_ERR_INVALID_ARG;
    if (dtype != FS_DTYPE_FP32 && dtype != FS_DTYPE_BF16 && dtype != FS_DTYPE_FP16) return FS_ERR_INVALID_ARG;
    if (!std::isfinite(eps) || eps < 0.0f) return FS_ERR_INVALID_ARG;
    if (rows == 0 || cols == 0) return FS_OK;
    if (!x || !y) return FS_ERR_INVALID_ARG;
    if (rows > (int64_t(1) << 40) || cols > (int64_t(1) << 40) || rows > (int64_t(1) << 60) / cols) return FS_ERR_INVALID_ARG;
    const int64_t bytes = rows * cols * elem_size(dtype);
    const char* xa = static_cast<const char*>(x);
    const char* ya = static_cast<const char*>(y);
    if (xa != ya && xa < ya + bytes && ya < xa + bytes) return FS_ERR_INVALID_ARG;      // partial overlap
    return FS_OK;
}

// ---------------------------------------------------------------------------------------------
// log_softmax
// ---------------------------------------------------------------------------------------------
template <int DT, int OUT> const void* lsm_warp_fn(const WarpGeom& g) {
    if (g.lanes == 32) {
        switch (g.vpl) {
            case 1: return (const void*)lsm_warp_kernel<DT, 32, 1, OUT>;
            case 2: return (const void*)lsm_warp_kernel<DT, 32, 2, OUT>;
            case 3: return (const void*)lsm_warp_kernel<DT, 32, 3, OUT>;
            case 4: return (const void*)lsm_warp_kernel<DT, 32, 4, OUT>;
            case 5: return (const void*)lsm_warp_kernel<DT, 32, 5, OUT>;
            case 6: return (const void*)lsm_warp_kernel<DT, 32, 6, OUT>;
            case 7: return (const void*)lsm_warp_kernel<DT, 32, 7, OUT>;
            case 8: return (const void*)lsm_warp_kernel<DT, 32, 8, OUT>;
            case 10: return (const void*)lsm_warp_long_kernel<DT, 10, OUT>;
            case 12: return (const void*)lsm_warp_long_kernel<DT, 12, OUT>;
            case 14: return (const void*)lsm_warp_long_kernel<DT, 14, OUT>;
            case 16: return (const void*)lsm_warp_long_kernel<DT, 16, OUT>;
            case 18: return (const void*)lsm_warp_long_kernel<DT, 18, OUT>;
            default: return nullptr;
        }
    }
    if (g.vpl == 1) return (const void*)lsm_warp_kernel<DT, 1, 1, OUT>;
    if (g.vpl == 2) return (const void*)lsm_warp_kernel<DT, 1, 2, OUT>;
    if (g.vpl != 4) return nullptr;
    switch (g.lanes) {
        case 1:  return (const void*)lsm_warp_kernel<DT, 1, 4, OUT>;
        case 2:  return (const void*)lsm_warp_kernel<DT, 2, 4, OUT>;
        case 4:  return (const void*)lsm_warp_kernel<DT, 4, 4, OUT>;
        case 8:  return (const void*)lsm_warp_kernel<DT, 8, 4, OUT>;
        default: return (const void*)lsm_warp_kernel<DT, 16, 4, OUT>;
    }
}

// out: OUT_LOG (log_softmax in x's dtype) or OUT_PROB32 (softmax of a 16-bit tensor written as binary32)
int run_log_softmax(const void* x, void* y, int64_t rows, int64_t cols, int dtype, float scale, int out, cudaStream_t st) {
    Device* devp = nullptr;
    int rc = get_device(&devp);
    if (rc != FS_OK) return rc;
    Device& dev = *devp;
    const int esz = elem_size(dtype);
    const bool fast = fast_path_ok(cols, dtype, ptr_align(x), ptr_align(y));
    LsmParams p{};
    p.x = x; p.y = y; p.rows = rows; p.cols = cols;
    p.nvec = fast ? cols * esz / 16 : 0;
    p.scale = std::fabs(scale);
    p.c = static_cast<float>(static_cast<double>(p.scale) * kLog2e);
    p.flip = std::signbit(scale) && scale != 0.0f ? (dtype == FS_DTYPE_FP32 ? 0x80000000u : 0x80008000u) : 0u;
    p.status = dev.status; p.pf_rows = 0;
    p.wide = (out == OUT_PROB32 && reinterpret_cast<uintptr_t>(y) % 32 == 0 && wide_store_enabled()) ? 1 : 0;   // (a row of y is a multiple of 32 bytes)
    if (fast && lsm_tile_wanted(dtype, p.nvec) && (out == OUT_LOG || dtype != FS_DTYPE_FP32)) {   // a warp per row from shared memory
        const void* fn = by_dtype(dtype, [&](auto dt) -> const void* {
            constexpr int DT = decltype(dt)::value;
            if constexpr (DT == DT_F32) return (const void*)lsm_tile_kernel<DT, OUT_LOG>;
            else return out == OUT_LOG ? (const void*)lsm_tile_kernel<DT, OUT_LOG> : (const void*)lsm_tile_kernel<DT, OUT_PROB32>; });
        const int t = 128;
        const size_t smem = size_t(t / 32) * size_t(p.nvec) * 16 + size_t(t / 32) * 8;
        int bps = 0;
        if ((rc = blocks_per_sm(dev, fn, t, smem, &bps)) != FS_OK) return rc;
        const int64_t grid = (rows + (t / 32) - 1) / (t / 32);
        if (grid <= 0x7fffffff) {
            p.pf_rows = prefetch_rows(dev.sm_count * bps) * (t / 32);
            set_first_wave_lag(p, dev.sm_count * bps, (t / 32) * p.nvec * 16);
            return launch(fn, grid, t, smem, 0, st, p);
        }
    }
    WarpGeom wg;
    bool warp_ok = fast && norm_warp_geom(p.nvec, dtype, &wg);
    if (fast && !warp_ok && p.nvec <= 576) {
        // rows of 4-9 KiB: still a warp per row (the row stays packed in registers: 10..18 vectors per lane);
        // the shared-memory kernel has too little to overlap on slices this short (measured 96-137 us
        // against 80 for a copy on 256 MiB)
        wg.lanes = 32; wg.vpl = static_cast<int>((p.nvec + 63) / 64) * 2; wg.r = 1;
        warp_ok = true;
    }
    if (warp_ok) {
        const void* fn = by_dtype(dtype, [&](auto dt) -> const void* {
            constexpr int DT = decltype(dt)::value;
            if constexpr (DT == DT_F32) return out == OUT_LOG ? lsm_warp_fn<DT, OUT_LOG>(wg) : nullptr;
            else return out == OUT_LOG ? lsm_warp_fn<DT, OUT_LOG>(wg) : lsm_warp_fn<DT, OUT_PROB32>(wg); });
        if (fn) {
            const int t = 128;
            const int64_t groups = (rows + (32 / wg.lanes) - 1) / (32 / wg.lanes);
            const int64_t grid = std::min<int64_t>((groups + (t / 32) - 1) / (t / 32), 0x7fffffff);
            return launch(fn, grid, t, 0, 0, st, p);
        }
    }
    SmemGeom sg;
    if (fast && dev.cluster_ok && smem_geom(p.nvec, dtype, 0, 0, &sg) && rows <= 0x7fffffff / sg.cs) {
        const bool full = smem_row_full(sg, dtype, p.nvec);
        // a ragged slice is padded with -inf, which a zero scale would turn into NaN: generic kernel
        if (full || p.c != 0.0f) {
            const void* fn = by_dtype(dtype, [&](auto dt) -> const void* {
                constexpr int DT = decltype(dt)::value;
                if constexpr (DT == DT_F32) {
                    return full ? (const void*)lsm_smem_kernel<DT, true, OUT_LOG> : (const void*)lsm_smem_kernel<DT, false, OUT_LOG>;
                } else {
                    if (out == OUT_LOG) return full ? (const void*)lsm_smem_kernel<DT, true, OUT_LOG> : (const void*)lsm_smem_kernel<DT, false, OUT_LOG>;
                    return full ? (const void*)lsm_smem_kernel<DT, true, OUT_PROB32> : (const void*)lsm_smem_kernel<DT, false, OUT_PROB32>;
                } });
            const size_t stage_bytes = smem_row_stage_bytes(sg, dtype);
            const size_t smem = stage_bytes + size_t(kNormMaxChunks) * 8;
            if (smem <= static_cast<size_t>(dev.smem_optin) - 2048) {
                int ncl = 0;
                if ((rc = active_clusters(dev, fn, sg.threads, smem, sg.cs, &ncl)) != FS_OK) return rc;
                p.pf_rows = prefetch_rows(ncl);
                set_first_wave_lag(p, ncl, p.nvec * 16);
                return launch(fn, rows * sg.cs, sg.threads, smem, sg.cs, st, p, static_cast<uint32_t>(stage_bytes), sg.slice,
                              smem_row_nchunk(sg, dtype));
            }
        }
    }
    const void* fn = by_dtype(dtype, [&](auto dt) -> const void* {
        constexpr int DT = decltype(dt)::value;
        if constexpr (DT == DT_F32) return (const void*)lsm_generic_kernel<DT, OUT_LOG>;
        else return out == OUT_LOG ? (const void*)lsm_generic_kernel<DT, OUT_LOG> : (const void*)lsm_generic_kernel<DT, OUT_PROB32>; });
    int t = 32;
    while (t < 1024 && cols > int64_t(t) * 8) t <<= 1;
    return launch(fn, std::min<int64_t>(rows, 0x7fffffff), t, 0, 0, st, p);
}

// ---------------------------------------------------------------------------------------------
// softmax backward
// ---------------------------------------------------------------------------------------------
template <int DT> const void* smb_warp_fn(const WarpGeom& g) {
    if (g.lanes == 32) {
        switch (g.vpl) {
            case 1: return (const void*)smb_warp_kernel<DT, 32, 1>;
            case 2: return (const void*)smb_warp_kernel<DT, 32, 2>;
            case 3: return (const void*)smb_warp_kernel<DT, 32, 3>;
            case 4: return (const void*)smb_warp_kernel<DT, 32, 4>;
            case 5: return (const void*)smb_warp_kernel<DT, 32, 5>;
            case 6: return (const void*)smb_warp_kernel<DT, 32, 6>;
            case 7: return (const void*)smb_warp_kernel<DT, 32, 7>;
            case 8: return (const void*)smb_warp_kernel<DT, 32, 8>;
            default: return nullptr;
        }
    }
    if (g.vpl == 1) return (const void*)smb_warp_kernel<DT, 1, 1>;
    if (g.vpl == 2) return (const void*)smb_warp_kernel<DT, 1, 2>;
    if (g.vpl != 4) return nullptr;
    switch (g.lanes) {
        case 1:  return (const void*)smb_warp_kernel<DT, 1, 4>;
        case 2:  return (const void*)smb_warp_kernel<DT, 2, 4>;
        case 4:  return (const void*)smb_warp_kernel<DT, 4, 4>;
        case 8:  return (const void*)smb_warp_kernel<DT, 8, 4>;
        default: return (const void*)smb_warp_kernel<DT, 16, 4>;
    }
}

int run_softmax_backward(const void* dy, const void* y, void* dx, int64_t rows, int64_t cols, int dtype, float scale,
                         cudaStream_t st) {
    Device* devp = nullptr;
    int rc = get_device(&devp);
    if (rc != FS_OK) return rc;
    Device& dev = *devp;
    const int esz = elem_size(dtype);
    const bool fast = fast_path_ok(cols, dtype, ptr_align(dy), ptr_align(y)) && ptr_align(dx) >= 16;
    SmbParams p{};
    p.dy = dy; p.y = y; p.dx = dx; p.rows = rows; p.cols = cols;
    p.nvec = fast ? cols * esz / 16 : 0;
    p.scale = scale; p.status = dev.status; p.pf_rows = 0;
    WarpGeom wg;
    if (fast && norm_warp_geom(p.nvec, dtype, &wg)) {
        const void* fn = by_dtype(dtype, [&](auto dt) -> const void* { return smb_warp_fn<decltype(dt)::value>(wg); });
        if (fn) {
            const int t = 128;
            const int64_t groups = (rows + (32 / wg.lanes) - 1) / (32 / wg.lanes);
            const int64_t grid = std::min<int64_t>((groups + (t / 32) - 1) / (t / 32), 0x7fffffff);
            return launch(fn, grid, t, 0, 0, st, p);
        }
    }
    if (fast && smb_tile_wanted(p.nvec)) {                  // rows of 4-8 KiB: a warp per row from shared memory
        const void* fn = by_dtype(dtype, [&](auto dt) -> const void* { return (const void*)smb_tile_kernel<decltype(dt)::value>; });
        const int t = 128;
        const size_t smem = 2 * size_t(t / 32) * size_t(p.nvec) * 16 + size_t(t / 32) * 8;
        int bps = 0;
        if ((rc = blocks_per_sm(dev, fn, t, smem, &bps)) != FS_OK) return rc;
        const int64_t grid = (rows + (t / 32) - 1) / (t / 32);
        if (grid <= 0x7fffffff) {
            p.pf_rows = prefetch_rows(dev.sm_count * bps) * (t / 32);
            set_first_wave_lag(p, dev.sm_count * bps, 2 * (t / 32) * p.nvec * 16);
            return launch(fn, grid, t, smem, 0, st, p);
        }
    }
    SmemGeom sg;
    if (fast && dev.cluster_ok && smem_geom(p.nvec, dtype, 0, 0, &sg) && rows <= 0x7fffffff / sg.cs) {
        const bool full = smem_row_full(sg, dtype, p.nvec);
        const void* fn = by_dtype(dtype, [&](auto dt) -> const void* {
            constexpr int DT = decltype(dt)::value;
            return full ? (const void*)smb_smem_kernel<DT, true> : (const void*)smb_smem_kernel<DT, false>; });
        const size_t stage_bytes = smem_row_stage_bytes(sg, dtype);
        const size_t smem = 2 * stage_bytes + size_t(kNormMaxChunks) * 8;      // the dy and the y slice
        if (smem <= static_cast<size_t>(dev.smem_optin) - 2048) {
            int ncl = 0;
            if ((rc = active_clusters(dev, fn, sg.threads, smem, sg.cs, &ncl)) != FS_OK) return rc;
            p.pf_rows = prefetch_rows(ncl);
            set_first_wave_lag(p, ncl, 2 * p.nvec * 16);
            return launch(fn, rows * sg.cs, sg.threads, smem, sg.cs, st, p, static_cast<uint32_t>(stage_bytes), sg.slice,
                          smem_row_nchunk(sg, dtype));
        }
    }
    const void* fn = by_dtype(dtype, [&](auto dt) -> const void* { return (const void*)smb_generic_kernel<decltype(dt)::value>; });
    int t = 32;
    while (t < 1024 && cols > int64_t(t) * 8) t <<= 1;
    return launch(fn, std::min<int64_t>(rows, 0x7fffffff), t, 0, 0, st, p);
}

// ---------------------------------------------------------------------------------------------
// softmax with an additive mask
// ---------------------------------------------------------------------------------------------
template <int DT> const void* masked_warp_fn(const WarpGeom& g) {
    if (g.lanes == 32) {
        switch (g.vpl) {
            case 1: return (const void*)sm_masked_warp_kernel<DT, 32, 1>;
            case 2: return (const void*)sm_masked_warp_kernel<DT, 32, 2>;
            case 3: return (const void*)sm_masked_warp_kernel<DT, 32, 3>;
            case 4: return (const void*)sm_masked_warp_kernel<DT, 32, 4>;
            case 5: return (const void*)sm_masked_warp_kernel<DT, 32, 5>;
            case 6: return (const void*)sm_masked_warp_kernel<DT, 32, 6>;
            case 7: return (const void*)sm_masked_warp_kernel<DT, 32, 7>;
            case 8: return (const void*)sm_masked_warp_kernel<DT, 32, 8>;
            case 10: return (const void*)sm_masked_warp_long_kernel<DT, 10>;
            case 12: return (const void*)sm_masked_warp_long_kernel<DT, 12>;
            case 14: return (const void*)sm_masked_warp_long_kernel<DT, 14>;
            case 16: return (const void*)sm_masked_warp_long_kernel<DT, 16>;
            case 18: return (const void*)sm_masked_warp_long_kernel<DT, 18>;
            default: return nullptr;
        }
    }
    if (g.vpl == 1) return (const void*)sm_masked_warp_kernel<DT, 1, 1>;
    if (g.vpl == 2) return (const void*)sm_masked_warp_kernel<DT, 1, 2>;
    if (g.vpl != 4) return nullptr;
    switch (g.lanes) {
        case 1:  return (const void*)sm_masked_warp_kernel<DT, 1, 4>;
        case 2:  return (const void*)sm_masked_warp_kernel<DT, 2, 4>;
        case 4:  return (const void*)sm_masked_warp_kernel<DT, 4, 4>;
        case 8:  return (const void*)sm_masked_warp_kernel<DT, 8, 4>;
        default: return (const void*)sm_masked_warp_kernel<DT, 16, 4>;
    }
}

// the four-rows-per-block kernel of fs_softmax_masked by number of batches (of 128 vectors) and whether the row fills them
template <int DT> const void* masked_tile_fn(int nb, bool full) {
    if constexpr (DT == DT_F32) {
        return nullptr;
    } else {
        switch (nb * 2 + (full ? 1 : 0)) {
            case 4:  return (const void*)sm_masked_tile_kernel<DT, 2, false>;
            case 5:  return (const void*)sm_masked_tile_kernel<DT, 2, true>;
            case 6:  return (const void*)sm_masked_tile_kernel<DT, 3, false>;
            case 7:  return (const void*)sm_masked_tile_kernel<DT, 3, true>;
            case 8:  return (const void*)sm_masked_tile_kernel<DT, 4, false>;
            case 9:  return (const void*)sm_masked_tile_kernel<DT, 4, true>;
            case 10: return (const void*)sm_masked_tile_kernel<DT, 5, false>;
            case 11: return (const void*)sm_masked_tile_kernel<DT, 5, true>;
            case 12: return (const void*)sm_masked_tile_kernel<DT, 6, false>;
            case 13: return (const void*)sm_masked_tile_kernel<DT, 6, true>;
            default: return nullptr;
        }
    }
}

int run_softmax_masked(const void* x, const void* mask, void* y, int64_t rows, int64_t cols, int64_t q_rows, int64_t heads,
                       int dtype, float scale, cudaStream_t st) {
    Device* devp = nullptr;
    int rc = get_device(&devp);
    if (rc != FS_OK) return rc;
    Device& dev = *devp;
    const int esz = elem_size(dtype);
    const bool fast = fast_path_ok(cols, dtype, ptr_align(x), ptr_align(y)) && ptr_align(mask) >= 16;
    MaskedParams p{};
    p.x = x; p.mask = mask; p.y = y; p.rows = rows; p.cols = cols;
    p.nvec = fast ? cols * esz / 16 : 0;
    p.q_rows = q_rows; p.group = q_rows * heads;
    p.c = static_cast<float>(static_cast<double>(scale) * kLog2e);
    p.status = dev.status; p.pf_rows = 0;
    if (fast && masked_tile_wanted(dtype, p.nvec)) {        // rows of 4-11 KiB: a warp per row from shared memory
        const int nb = static_cast<int>((p.nvec + 127) / 128);          // batches of 4 vectors per lane
        const bool full = p.nvec % 128 == 0;
        const void* fn = by_dtype(dtype, [&](auto dt) -> const void* { return masked_tile_fn<decltype(dt)::value>(nb, full); });
        const int t = 128;
        const size_t smem = size_t(t / 32) * size_t(p.nvec) * 16 + size_t(t / 32) * 8;
        const int64_t grid = (rows + (t / 32) - 1) / (t / 32);
        if (fn && grid <= 0x7fffffff) {                     // (a forced range beyond six batches goes to the kernels below)
            int bps = 0;
            if ((rc = blocks_per_sm(dev, fn, t, smem, &bps)) != FS_OK) return rc;
            p.pf_rows = prefetch_rows(dev.sm_count * bps) * (t / 32);
            set_first_wave_lag(p, dev.sm_count * bps, (t / 32) * p.nvec * 16);
            return launch(fn, grid, t, smem, 0, st, p);
        }
    }
    WarpGeom wg;
    bool warp_ok = fast && norm_warp_geom(p.nvec, dtype, &wg);
    if (fast && !warp_ok && p.nvec <= 576) {        // rows of 4-9 KiB: still a warp per row, 10..18 packed vectors per lane
        wg.lanes = 32; wg.vpl = static_cast<int>((p.nvec + 63) / 64) * 2; wg.r = 1;
        warp_ok = true;
    }
    if (warp_ok) {
        const void* fn = by_dtype(dtype, [&](auto dt) -> const void* { return masked_warp_fn<decltype(dt)::value>(wg); });
        if (fn) {
            const int t = 128;
            const int64_t groups = (rows + (32 / wg.lanes) - 1) / (32 / wg.lanes);
            const int64_t grid = std::min<int64_t>((groups + (t / 32) - 1) / (t / 32), 0x7fffffff);
            return launch(fn, grid, t, 0, 0, st, p);
        }
    }
    SmemGeom sg;
    if (fast && dev.cluster_ok && smem_geom(p.nvec, dtype, 0, 0, &sg) && rows <= 0x7fffffff / sg.cs) {
        const bool full = smem_row_full(sg, dtype, p.nvec);
        const void* fn = by_dtype(dtype, [&](auto dt) -> const void* {
            constexpr int DT = decltype(dt)::value;
            return full ? (const void*)sm_masked_smem_kernel<DT, true> : (const void*)sm_masked_smem_kernel<DT, false>; });
        const size_t stage_bytes = smem_row_stage_bytes(sg, dtype);
        const size_t smem = stage_bytes + size_t(kNormMaxChunks) * 8 + size_t(2 * kNormMaxChunks) * sg.threads * 4;
        if (smem <= static_cast<size_t>(dev.smem_optin) - 2048) {
            int ncl = 0;
            if ((rc = active_clusters(dev, fn, sg.threads, smem, sg.cs, &ncl)) != FS_OK) return rc;
            p.pf_rows = prefetch_rows(ncl);
            set_first_wave_lag(p, ncl, p.nvec * 16);
            return launch(fn, rows * sg.cs, sg.threads, smem, sg.cs, st, p, static_cast<uint32_t>(stage_bytes), sg.slice,
                          smem_row_nchunk(sg, dtype));
        }
    }
    const void* fn = by_dtype(dtype, [&](auto dt) -> const void* { return (const void*)sm_masked_generic_kernel<decltype(dt)::value>; });
    int t = 32;
    while (t < 1024 && cols > int64_t(t) * 8) t <<= 1;
    return launch(fn, std::min<int64_t>(rows, 0x7fffffff), t, 0, 0, st, p);
}

}  // namespace

extern "C" {

int fs_softmax_ex(const void* x, void* y, int64_t rows, int64_t cols, int dtype, float scale,
                  void* stream, int kernel, int threads, int cluster) {
    const int v = validate(x, y, rows, cols, dtype, scale);
    if (v != FS_OK) return v;
    if (kernel < FS_KERNEL_AUTO || kernel > FS_KERNEL_GENERIC) return FS_ERR_INVALID_ARG;
    if (cluster < 0 || cluster > kMaxCluster) return FS_ERR_INVALID_ARG;
    if (rows == 0 || cols == 0) return FS_OK;
    FS_CHECK_PTRS(x, y);
    FS_DBG_RANGES({x, (unsigned long long)(rows * cols * elem_size(dtype)), 0}, {y, (unsigned long long)(rows * cols * elem_size(dtype)), 1});
    return run(x, y, rows, cols, dtype, scale, static_cast<cudaStream_t>(stream), kernel, threads, cluster);
}

int fs_softmax(const void* x, void* y, int64_t rows, int64_t cols, int dtype, float scale, void* stream) {
    return fs_softmax_ex(x, y, rows, cols, dtype, scale, stream, FS_KERNEL_AUTO, 0, 0);
}

int fs_softmax_causal(const void* x, void* y, int64_t rows, int64_t cols, int64_t q_offset, int dtype, float scale,
                      void* stream) {
    const int v = validate(x, y, rows, cols, dtype, scale);
    if (v != FS_OK) return v;
    if (rows == 0 || cols == 0) return FS_OK;
    if (q_offset > (int64_t(1) << 41) || q_offset < -(int64_t(1) << 41)) return FS_ERR_INVALID_ARG;
    FS_CHECK_PTRS(x, y);
    FS_DBG_RANGES({x, (unsigned long long)(rows * cols * elem_size(dtype)), 0}, {y, (unsigned long long)(rows * cols * elem_size(dtype)), 1});
    return run_causal(x, y, rows, cols, q_offset, dtype, scale, static_cast<cudaStream_t>(stream));
}

int fs_router_topk(const void* x, float* w, int32_t* idx, int64_t rows, int64_t cols, int k, int dtype, float scale,
                   int renormalize, void* stream) {
    if (rows < 0 || cols < 0) return FS_ERR_INVALID_ARG;
    if (dtype != FS_DTYPE_FP32 && dtype != FS_DTYPE_BF16 && dtype != FS_DTYPE_FP16) return FS_ERR_INVALID_ARG;
    if (!std::isfinite(scale)) return FS_ERR_INVALID_ARG;
    if (rows == 0) return FS_OK;
    if (k < 1 || k > cols || k > FS_ROUTER_MAX_K) return FS_ERR_INVALID_ARG;
    if (!x || !w || !idx) return FS_ERR_INVALID_ARG;
    if (rows > (int64_t(1) << 40)) return FS_ERR_INVALID_ARG;
    if (ptr_align(x) < 16 || (cols * elem_size(dtype)) % 16 != 0) return FS_ERR_UNSUPPORTED;
    if (ptr_align(w) < 4 || ptr_align(idx) < 4) return FS_ERR_INVALID_ARG;
    FS_CHECK_PTRS(x, w, idx);
    FS_DBG_RANGES({x, (unsigned long long)(rows * cols * elem_size(dtype)), 0}, {w, (unsigned long long)(rows * k * 4), 1}, {idx, (unsigned long long)(rows * k * 4), 1});
    const int64_t nvec = cols * elem_size(dtype) / 16;
    WarpGeom g;
    if (!warp_geom(nvec, dtype, &g) || g.vpl * (dtype == FS_DTYPE_FP32 ? 4 : 8) > 32) return FS_ERR_UNSUPPORTED;
    Device* dev = nullptr;
    int rc = get_device(&dev);
    if (rc != FS_OK) return rc;
    // k <= 8 selects with sorting networks in registers (FS_ROUTER_ROUNDS=1, read once, keeps the
    // kernel that takes one maximum per round, which serves any k)
    static const bool rounds_only = env_int("FS_ROUTER_ROUNDS", 0) != 0;
    const bool net = k <= 8 && !rounds_only;
    const bool full = nvec == int64_t(g.lanes) * g.vpl;        // no padding vectors in a row's lanes
    const void* fn = nullptr;
    switch (dtype) {
        case FS_DTYPE_FP32: fn = net ? router8_fn<DT_F32>(g, full) : router_fn<DT_F32>(g); break;
        case FS_DTYPE_BF16: fn = net ? router8_fn<DT_BF16>(g, full) : router_fn<DT_BF16>(g); break;
        default:            fn = net ? router8_fn<DT_F16>(g, full) : router_fn<DT_F16>(g); break;
    }
    if (!fn) return FS_ERR_UNSUPPORTED;
    RouterParams p;
    p.x = x; p.w = w; p.idx = idx; p.rows = rows; p.nvec = nvec; p.k = k;
    p.c = static_cast<float>(static_cast<double>(scale) * kLog2e);
    p.renorm = renormalize ? 1 : 0;
    p.wide = (net && k == 8 && reinterpret_cast<uintptr_t>(w) % 32 == 0 && reinterpret_cast<uintptr_t>(idx) % 32 == 0 && wide_store_enabled()) ? 1 : 0;
    const int t = 128;
    const size_t smem = net ? 0 : static_cast<size_t>(g.vpl) * (dtype == FS_DTYPE_FP32 ? 4 : 8) * t * sizeof(uint32_t);   // <= 16 KiB
    const int64_t groups = (rows + (32 / g.lanes) - 1) / (32 / g.lanes);
    const int64_t grid = std::min<int64_t>((groups + (t / 32) - 1) / (t / 32), 0x7fffffff);
    return launch(fn, grid, t, smem, 0, static_cast<cudaStream_t>(stream), p);
}

int fs_log_softmax(const void* x, void* y, int64_t rows, int64_t cols, int dtype, float scale, void* stream) {
    const int v = validate(x, y, rows, cols, dtype, scale);
    if (v != FS_OK) return v;
    if (rows == 0 || cols == 0) return FS_OK;
    FS_CHECK_PTRS(x, y);
    FS_DBG_RANGES({x, (unsigned long long)(rows * cols * elem_size(dtype)), 0}, {y, (unsigned long long)(rows * cols * elem_size(dtype)), 1});
    return run_log_softmax(x, y, rows, cols, dtype, scale, OUT_LOG, static_cast<cudaStream_t>(stream));
}

int fs_softmax_masked(const void* x, const void* mask, void* y, int64_t rows, int64_t cols, int64_t q_rows, int64_t heads,
                      int dtype, float scale, void* stream) {
    const int v = validate(x, y, rows, cols, dtype, scale);
    if (v != FS_OK) return v;
    if (q_rows < 1 || heads < 1 || q_rows > (int64_t(1) << 40) || heads > (int64_t(1) << 20)) return FS_ERR_INVALID_ARG;
    if (rows % (q_rows * heads) != 0) return FS_ERR_INVALID_ARG;
    if (rows == 0 || cols == 0) return FS_OK;
    if (!mask) return FS_ERR_INVALID_ARG;
    FS_CHECK_PTRS(x, mask, y);
    FS_DBG_RANGES({x, (unsigned long long)(rows * cols * elem_size(dtype)), 0}, {mask, (unsigned long long)(rows / heads * cols * elem_size(dtype)), 0},
                  {y, (unsigned long long)(rows * cols * elem_size(dtype)), 1});
    return run_softmax_masked(x, mask, y, rows, cols, q_rows, heads, dtype, scale, static_cast<cudaStream_t>(stream));
}

int fs_softmax_backward(const void* dy, const void* y, void* dx, int64_t rows, int64_t cols, int dtype, float scale,
                        void* stream) {
    int v = validate(dy, dx, rows, cols, dtype, scale);
    if (v == FS_OK) v = validate(y, dx, rows, cols, dtype, scale);
    if (v != FS_OK) return v;
    if (rows == 0 || cols == 0) return FS_OK;
    FS_CHECK_PTRS(dy, y, dx);
    FS_DBG_RANGES({dy, (unsigned long long)(rows * cols * elem_size(dtype)), 0}, {y, (unsigned long long)(rows * cols * elem_size(dtype)), 0},
                  {dx, (unsigned long long)(rows * cols * elem_size(dtype)), 1});
    return run_softmax_backward(dy, y, dx, rows, cols, dtype, scale, static_cast<cudaStream_t>(stream));
}

int fs_softmax_f32out(const void* x, float* y, int64_t rows, int64_t cols, int dtype, float scale, void* stream) {
    if (rows < 0 || cols < 0 || !std::isfinite(scale)) return FS_ERR_INVALID_ARG;
    if (dtype != FS_DTYPE_BF16 && dtype != FS_DTYPE_FP16) return FS_ERR_INVALID_ARG;
    if (rows == 0 || cols == 0) return FS_OK;
    if (!x || !y) return FS_ERR_INVALID_ARG;
    if (cols > (int64_t(1) << 40) || rows > (int64_t(1) << 40) || rows > (int64_t(1) << 59) / cols) return FS_ERR_INVALID_ARG;
    if (ptr_align(y) < 4) return FS_ERR_INVALID_ARG;
    const uintptr_t a = reinterpret_cast<uintptr_t>(x), b = reinterpret_cast<uintptr_t>(y);
    const uintptr_t na = static_cast<uintptr_t>(rows * cols * 2), nb = static_cast<uintptr_t>(rows * cols * 4);
    if (a < b + nb && b < a + na) return FS_ERR_INVALID_ARG;          // the tensors differ in size: no overlap at all
    FS_CHECK_PTRS(x, y);
    FS_DBG_RANGES({x, (unsigned long long)(rows * cols * 2), 0}, {y, (unsigned long long)(rows * cols * 4), 1});
    return run_log_softmax(x, y, rows, cols, dtype, scale, OUT_PROB32, static_cast<cudaStream_t>(stream));
}

int fs_layer_norm(const void* x, const void* gamma, const void* beta, void* y, int64_t rows, int64_t cols, int dtype,
                  float eps, void* stream) {
    const int v = validate_norm(x, y, rows, cols, dtype, eps);
    if (v != FS_OK || rows == 0 || cols == 0) return v;
    const int aff = (gamma || beta) ? 1 : 0;
    FS_CHECK_PTRS(x, gamma, beta, y);
    FS_DBG_RANGES({x, (unsigned long long)(rows * cols * elem_size(dtype)), 0}, {gamma, (unsigned long long)(cols * elem_size(dtype)), 0},
                  {beta, (unsigned long long)(cols * elem_size(dtype)), 0}, {y, (unsigned long long)(rows * cols * elem_size(dtype)), 1});
    return run_norm(x, gamma, beta, y, rows, cols, dtype, eps, aff, 1, 1, static_cast<cudaStream_t>(stream));
}

int fs_group_norm(const void* x, const void* gamma, const void* beta, void* y, int64_t n, int64_t channels, int64_t spatial,
                  int64_t groups, int dtype, float eps, void* stream) {
    if (n < 0 || channels < 0 || spatial < 0 || groups < 1 || channels % groups != 0) return FS_ERR_INVALID_ARG;
    if (channels > (int64_t(1) << 30) || spatial > (int64_t(1) << 40) || n > (int64_t(1) << 40) / groups) return FS_ERR_INVALID_ARG;
    const int64_t rows = n * groups;
    const int64_t cpg = channels / groups;
    if (cpg > 0 && spatial > (int64_t(1) << 40) / cpg) return FS_ERR_INVALID_ARG;
    const int64_t cols = cpg * spatial;
    const int v = validate_norm(x, y, rows, cols, dtype, eps);
    if (v != FS_OK || rows == 0 || cols == 0) return v;
    const int aff = (gamma || beta) ? 2 : 0;
    FS_CHECK_PTRS(x, gamma, beta, y);
    FS_DBG_RANGES({x, (unsigned long long)(rows * cols * elem_size(dtype)), 0}, {gamma, (unsigned long long)(channels * elem_size(dtype)), 0},
                  {beta, (unsigned long long)(channels * elem_size(dtype)), 0}, {y, (unsigned long long)(rows * cols * elem_size(dtype)), 1});
    return run_norm(x, gamma, beta, y, rows, cols, dtype, eps, aff, spatial, groups, static_cast<cudaStream_t>(stream));
}

int fs_split_geometry(int64_t cols, int dtype, int* cluster, int* threads, int64_t* slice_bytes) {
    if (cols < 1 || !cluster || !threads || !slice_bytes) return FS_ERR_INVALID_ARG;
    if (dtype != FS_DTYPE_FP32 && dtype != FS_DTYPE_BF16 && dtype != FS_DTYPE_FP16) return FS_ERR_INVALID_ARG;
    if (cols > (int64_t(1) << 40) || (cols * elem_size(dtype)) % 16 != 0) return FS_ERR_UNSUPPORTED;
    SmemGeom g;
    if (!smem_geom(cols * elem_size(dtype) / 16, dtype, 0, 0, &g)) return FS_ERR_UNSUPPORTED;
    *cluster = g.cs; *threads = g.threads; *slice_bytes = int64_t(g.slice) * 16;
    return FS_OK;
}

int fs_select_kernel(int64_t rows, int64_t cols, int dtype, int x_align, int y_align) {
    if (rows < 0 || cols < 0 || x_align < 1 || y_align < 1) return -FS_ERR_INVALID_ARG;
    if (dtype != FS_DTYPE_FP32 && dtype != FS_DTYPE_BF16 && dtype != FS_DTYPE_FP16) return -FS_ERR_INVALID_ARG;
    return select_kernel(cols, dtype, x_align, y_align);
}

int fs_copy(const void* x, void* y, int64_t bytes, void* stream) {
    if (bytes < 0 || bytes % 16) return FS_ERR_INVALID_ARG;
    if (bytes == 0) return FS_OK;
    if (!x || !y || ptr_align(x) < 16 || ptr_align(y) < 16) return FS_ERR_INVALID_ARG;
    FS_CHECK_PTRS(x, y);
    FS_DBG_RANGES({x, (unsigned long long)bytes, 0}, {y, (unsigned long long)bytes, 1});
    Device* dev = nullptr;
    int rc = get_device(&dev);
    if (rc != FS_OK) return rc;
    const void* fn = (const void*)copy_kernel;
    const int64_t nvec = bytes / 16;
    const int64_t grid = std::min<int64_t>((nvec + 1023) / 1024, 0x7fffffff);
    const uint4* xv = static_cast<const uint4*>(x);
    uint4* yv = static_cast<uint4*>(y);
    return launch(fn, grid, 256, 0, 0, static_cast<cudaStream_t>(stream), xv, yv, nvec, int(early_prefetch_enabled()));
}

int fs_softmax_host(const void* x_host, void* y_host, int64_t rows, int64_t cols, int dtype, float scale) {
    const int v = validate(x_host, y_host, rows, cols, dtype, scale);
    if (v != FS_OK) return v;
    if (rows == 0 || cols == 0) return FS_OK;
    Device* devp = nullptr;
    int rc = get_device(&devp);
    if (rc != FS_OK) return rc;
    Device& dev = *devp;
    std::lock_guard<std::mutex> lk(g_host_mu);
#ifdef FS_DEBUG_BOUNDS
    t_dbg = DebugRanges{};              // the staging buffers are the library's own: unchecked
#endif

    const size_t row_bytes = static_cast<size_t>(cols) * elem_size(dtype);
    // chunk size: small enough that filling and draining the pipeline costs little, large enough
    // that the ~10 runtime calls per chunk (20 us of host time) stay hidden behind the copies;
    // 8 MiB measured best on PCIe Gen5 (FS_HOST_CHUNK_MB overrides, for tuning)
    static const size_t chunk_mb = [] { const char* e = std::getenv("FS_HOST_CHUNK_MB"); int v = e ? std::atoi(e) : 0; return size_t(v > 0 ? v : 8); }();
    const size_t target = chunk_mb << 20;
    int64_t chunk_rows = std::max<int64_t>(1, static_cast<int64_t>(target / row_bytes));
    chunk_rows = std::min<int64_t>(chunk_rows, rows);
    const size_t need = (static_cast<size_t>(chunk_rows) * row_bytes + 255) / 256 * 256;
    if (need > dev.slot_bytes) {
        for (int s = 0; s < Device::kSlots; ++s) {
            if (dev.dx[s]) FS_CUDA(cudaFree(dev.dx[s]));
            if (dev.dy[s]) FS_CUDA(cudaFree(dev.dy[s]));
            dev.dx[s] = dev.dy[s] = nullptr;
        }
        dev.slot_bytes = 0;
        for (int s = 0; s < Device::kSlots; ++s) {
            FS_CUDA(cudaMalloc(&dev.dx[s], need));
            FS_CUDA(cudaMalloc(&dev.dy[s], need));
        }
        dev.slot_bytes = need;
    }
    if (!dev.s_in) {
        FS_CUDA(cudaStreamCreateWithFlags(&dev.s_in, cudaStreamNonBlocking));
        FS_CUDA(cudaStreamCreateWithFlags(&dev.s_run, cudaStreamNonBlocking));
        FS_CUDA(cudaStreamCreateWithFlags(&dev.s_out, cudaStreamNonBlocking));
        for (int s = 0; s < Device::kSlots; ++s) {
            FS_CUDA(cudaEventCreateWithFlags(&dev.ev_in[s], cudaEventDisableTiming));
            FS_CUDA(cudaEventCreateWithFlags(&dev.ev_run[s], cudaEventDisableTiming));
            FS_CUDA(cudaEventCreateWithFlags(&dev.ev_out[s], cudaEventDisableTiming));
        }
    }

    // Three streams, one per stage: copies in run back to back on the host-to-device engine,
    // kernels on the SMs, copies out on the device-to-host engine. Events hand a slot from stage
    // to stage and back (a slot's input buffer is free once its kernel ran, its output buffer once
    // it was copied out), so the stages overlap across chunks.
    const char* xin = static_cast<const char*>(x_host);
    char* yout = static_cast<char*>(y_host);
    int slot = 0;
    int64_t chunk = 0;
    for (int64_t r0 = 0; r0 < rows; r0 += chunk_rows, slot = (slot + 1) % Device::kSlots, ++chunk) {
        const int64_t nr = std::min<int64_t>(chunk_rows, rows - r0);
        const size_t bytes = static_cast<size_t>(nr) * row_bytes;
        if (chunk >= Device::kSlots) FS_CUDA(cudaStreamWaitEvent(dev.s_in, dev.ev_run[slot], 0));
        FS_CUDA(cudaMemcpyAsync(dev.dx[slot], xin + static_cast<size_t>(r0) * row_bytes, bytes, cudaMemcpyHostToDevice, dev.s_in));
        FS_CUDA(cudaEventRecord(dev.ev_in[slot], dev.s_in));
        FS_CUDA(cudaStreamWaitEvent(dev.s_run, dev.ev_in[slot], 0));
        if (chunk >= Device::kSlots) FS_CUDA(cudaStreamWaitEvent(dev.s_run, dev.ev_out[slot], 0));
        rc = run(dev.dx[slot], dev.dy[slot], nr, cols, dtype, scale, dev.s_run, FS_KERNEL_AUTO, 0, 0);
        if (rc != FS_OK) return rc;
        FS_CUDA(cudaEventRecord(dev.ev_run[slot], dev.s_run));
        FS_CUDA(cudaStreamWaitEvent(dev.s_out, dev.ev_run[slot], 0));
        FS_CUDA(cudaMemcpyAsync(yout + static_cast<size_t>(r0) * row_bytes, dev.dy[slot], bytes, cudaMemcpyDeviceToHost, dev.s_out));
        FS_CUDA(cudaEventRecord(dev.ev_out[slot], dev.s_out));
    }
    FS_CUDA(cudaStreamSynchronize(dev.s_out));
    FS_CUDA(cudaStreamSynchronize(dev.s_run));
    FS_CUDA(cudaStreamSynchronize(dev.s_in));
    return FS_OK;
}

int fs_release(void) {
    int d = 0;
    FS_CUDA(cudaGetDevice(&d));
    if (d < 0 || d >= kMaxDevices) return FS_ERR_UNSUPPORTED;
    std::lock_guard<std::mutex> lk(g_host_mu);
    Device& dev = g_dev[d];
    cudaStream_t* streams[3] = {&dev.s_in, &dev.s_run, &dev.s_out};
    for (cudaStream_t* st : streams) {
        if (*st) { FS_CUDA(cudaStreamSynchronize(*st)); FS_CUDA(cudaStreamDestroy(*st)); *st = nullptr; }
    }
    for (int s = 0; s < Device::kSlots; ++s) {
        if (dev.ev_in[s]) { FS_CUDA(cudaEventDestroy(dev.ev_in[s])); dev.ev_in[s] = nullptr; }
        if (dev.ev_run[s]) { FS_CUDA(cudaEventDestroy(dev.ev_run[s])); dev.ev_run[s] = nullptr; }
        if (dev.ev_out[s]) { FS_CUDA(cudaEventDestroy(dev.ev_out[s])); dev.ev_out[s] = nullptr; }
        if (dev.dx[s]) { FS_CUDA(cudaFree(dev.dx[s])); dev.dx[s] = nullptr; }
        if (dev.dy[s]) { FS_CUDA(cudaFree(dev.dy[s])); dev.dy[s] = nullptr; }
    }
    dev.slot_bytes = 0;
    {
        std::lock_guard<std::mutex> sl(g_scratch_mu);
        if (dev.scratch) {
            FS_CUDA(cudaDeviceSynchronize());
            FS_CUDA(cudaFree(dev.scratch));
            dev.scratch = nullptr; dev.scratch_bytes = 0; dev.scratch_used = false;
        }
        if (dev.scratch_ev) { FS_CUDA(cudaEventDestroy(dev.scratch_ev)); dev.scratch_ev = nullptr; }
    }
    return FS_OK;
}

int fs_device_status(void) {
    Device* dev = nullptr;
    int rc = get_device(&dev);
    if (rc != FS_OK) return rc;
    int word = 0;
    FS_CUDA(cudaDeviceSynchronize());
    FS_CUDA(cudaMemcpy(&word, dev->status, sizeof(int), cudaMemcpyDeviceToHost));
    if (word) FS_CUDA(cudaMemset(dev->status, 0, sizeof(int)));
#ifdef FS_DEBUG_BOUNDS
    {
        int flags = 0, zero = 0;
        FS_CUDA(cudaMemcpyFromSymbol(&flags, g_dbg, sizeof(int), offsetof(DebugRanges, flags)));
        if (flags) FS_CUDA(cudaMemcpyToSymbol(g_dbg, &zero, sizeof(int), offsetof(DebugRanges, flags)));
        word |= flags;
    }
#endif
    if (word & DEV_BOUNDS) return FS_ERR_DEVICE_BOUNDS;
    return (word & DEV_TIMEOUT) ? FS_ERR_DEVICE_TIMEOUT : FS_OK;
}

int fs_debug_checked_build(void) {
#ifdef FS_DEBUG_BOUNDS
    return 1;
#else
    return 0;
#endif
}

int fs_debug_shrink_writable(int64_t bytes) {
#ifdef FS_DEBUG_BOUNDS
    t_dbg_shrink = bytes > 0 ? bytes : 0;
    return FS_OK;
#else
    (void)bytes;
    return FS_ERR_UNSUPPORTED;
#endif
}

int fs_debug_bad_address(uint64_t* address) {
    if (!address) return FS_ERR_INVALID_ARG;
    *address = 0;
#ifdef FS_DEBUG_BOUNDS
    unsigned long long bad = 0, zero = 0;
    FS_CUDA(cudaDeviceSynchronize());
    FS_CUDA(cudaMemcpyFromSymbol(&bad, g_dbg, sizeof(bad), offsetof(DebugRanges, first_bad)));
    if (bad) FS_CUDA(cudaMemcpyToSymbol(g_dbg, &zero, sizeof(zero), offsetof(DebugRanges, first_bad)));
    *address = bad;
    return FS_OK;
#else
    return FS_ERR_UNSUPPORTED;
#endif
}

int fs_softmax_static(const void* x, void* y, int64_t rows, int64_t cols, int dtype, float scale, void* stream) {
    const int v = validate(x, y, rows, cols, dtype, scale);
    if (v != FS_OK) return v;
    if (rows == 0 || cols == 0) return FS_OK;
    if (!fast_path_ok(cols, dtype, ptr_align(x), ptr_align(y))) return FS_ERR_UNSUPPORTED;
    const int64_t nvec = cols * elem_size(dtype) / 16;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
#ifdef FS_DEBUG_BOUNDS
    t_dbg = DebugRanges{};              // fs_static_status does not read the checker's flag word: this entry point goes unchecked
#endif
    std::lock_guard<std::mutex> lk(g_static_mu);
    StaticDevice* sdp = nullptr;
    int rc = get_static_device(&sdp);
    if (rc != FS_OK) return rc;
    StaticDevice& sd = *sdp;

    SmemGeom sg;
    if (!smem_geom(nvec, dtype, 0, 0, &sg)) {
        // rows beyond FS_STATIC_MAX_ROW_BYTES: the two-kernel path, its pairs in the array
        SplitPlan sp;
        if (!softmax_split_plan(sd.sm_count, sd.scratch, x, y, rows, cols, dtype, scale, &sp)) return FS_ERR_UNSUPPORTED;
        if (rows * sp.nseg > FS_STATIC_MAX_PAIRS) return FS_ERR_UNSUPPORTED;      // more pairs than the array holds
        return softmax_split_launch(sp, dtype, reinterpret_cast<float2*>(sd.scratch + kStaticPairOffsetWords), st);
    }
    if (rows > 0x7fffffff / sg.cs) return FS_ERR_UNSUPPORTED;
    if (!sd.cluster_ok) return FS_ERR_UNSUPPORTED;

    Params p{};
    p.x = x; p.y = y; p.rows = rows; p.cols = cols; p.nvec = nvec;
    p.c = static_cast<float>(static_cast<double>(scale) * kLog2e);
    p.neg = p.c < 0.0f ? 1 : 0;
    p.status = sd.scratch;
    p.q_offset = 0;
    p.pf_rows = 0;
    p.wait_polls = kDefaultWaitPolls;
    p.early_pf = early_prefetch_enabled();
    const void* fn = smem_row_fn(dtype, p.neg, sg, nvec);
    const size_t stage_bytes = smem_row_stage_bytes(sg, dtype);
    const size_t smem = smem_row_bytes(sg, dtype);
    if (smem > static_cast<size_t>(sd.smem_optin) - 2048) return FS_ERR_UNSUPPORTED;
    if (p.c == 0.0f && !smem_row_full(sg, dtype, nvec)) return FS_ERR_UNSUPPORTED;   // see the header
    const bool full_variant = smem_row_full(sg, dtype, nvec);
    if (!sd.configured[dtype][p.neg][full_variant]) {
        cudaFuncAttributes fa;
        FS_CUDA(cudaFuncGetAttributes(&fa, fn));
        FS_CUDA(cudaFuncSetAttribute(fn, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                     sd.smem_optin - static_cast<int>(fa.sharedSizeBytes)));
        FS_CUDA(cudaFuncSetAttribute(fn, cudaFuncAttributeNonPortableClusterSizeAllowed, 1));
        sd.configured[dtype][p.neg][full_variant] = true;
    }
    int ncl = 0;
    for (int i = 0; i < sd.ngeo && !ncl; ++i)
        if (sd.geo[i].fn == fn && sd.geo[i].threads == sg.threads && sd.geo[i].cs == sg.cs && sd.geo[i].smem == smem) ncl = sd.geo[i].ncl;
    if (!ncl) {
        cudaLaunchConfig_t cfg = {};
        cfg.gridDim = dim3(sg.cs * sd.sm_count, 1, 1);
        cfg.blockDim = dim3(sg.threads, 1, 1);
        cfg.dynamicSmemBytes = smem;
        cudaLaunchAttribute attr[1];
        attr[0].id = cudaLaunchAttributeClusterDimension;
        attr[0].val.clusterDim.x = sg.cs; attr[0].val.clusterDim.y = 1; attr[0].val.clusterDim.z = 1;
        cfg.attrs = attr; cfg.numAttrs = 1;
        FS_CUDA(cudaOccupancyMaxActiveClusters(&ncl, fn, &cfg));
        if (ncl < 1) return FS_ERR_UNSUPPORTED;
        if (sd.ngeo < 16) sd.geo[sd.ngeo++] = StaticDevice::Geo{fn, sg.threads, sg.cs, smem, ncl};
    }
    p.pf_rows = prefetch_rows(ncl);
    set_first_wave_lag(p, ncl, nvec * 16);
    return launch(fn, rows * sg.cs, sg.threads, smem, sg.cs, st, p,
                  static_cast<uint32_t>(stage_bytes), sg.slice, smem_row_nchunk(sg, dtype));
}

int fs_static_status(void) {
    std::lock_guard<std::mutex> lk(g_static_mu);
    StaticDevice* sd = nullptr;
    int rc = get_static_device(&sd);
    if (rc != FS_OK) return rc;
    int word = 0;
    FS_CUDA(cudaDeviceSynchronize());
    FS_CUDA(cudaMemcpy(&word, sd->scratch, sizeof(int), cudaMemcpyDeviceToHost));
    if (word) FS_CUDA(cudaMemset(sd->scratch, 0, sizeof(int)));
    return (word & DEV_TIMEOUT) ? FS_ERR_DEVICE_TIMEOUT : FS_OK;
}

// ---- self-tests of the bounded waits (nothing here can fault or hang a device) -------------------

int fs_debug_set_wait_polls(int polls) {
    Device* dev = nullptr;
    int rc = get_device(&dev);
    if (rc != FS_OK) return rc;
    dev->wait_polls.store(polls > 0 ? polls : kDefaultWaitPolls, std::memory_order_relaxed);
    return FS_OK;
}

int fs_debug_wait_probe(void* stream) {
    Device* dev = nullptr;
    int rc = get_device(&dev);
    if (rc != FS_OK) return rc;
    return launch((const void*)wait_probe_kernel, 1, 64, 0, 0, static_cast<cudaStream_t>(stream), dev->status,
                  dev->wait_polls.load(std::memory_order_relaxed));
}

int fs_debug_softmax_expire(const void* x, void* y, int64_t rows, int64_t cols, int dtype, float scale, void* stream,
                            int threads, int cluster) {
    const int v = validate(x, y, rows, cols, dtype, scale);
    if (v != FS_OK) return v;
    if (cluster < 0 || cluster > kMaxCluster) return FS_ERR_INVALID_ARG;
    if (rows == 0 || cols == 0) return FS_OK;
    // every chunk barrier of the split-row kernel is armed for 16 bytes more than are copied
    return run(x, y, rows, cols, dtype, scale, static_cast<cudaStream_t>(stream), FS_KERNEL_CLUSTER, threads, cluster, 16u);
}

int fs_last_cuda_error(void) { return t_last_cuda_error; }

const char* fs_strerror(int status) {
    switch (status) {
        case FS_OK: return "ok";
        case FS_ERR_INVALID_ARG: return "invalid argument";
        case FS_ERR_UNSUPPORTED: return "unsupported shape, alignment or launch geometry for the requested kernel";
        case FS_ERR_CUDA: return "CUDA error (see fs_last_cuda_error)";
        case FS_ERR_DEVICE_TIMEOUT: return "a bounded device-side wait expired";
        case FS_ERR_DEVICE_BOUNDS: return "checked build: a kernel tried to access memory outside the tensors of its call (the access was skipped)";
        default: return "unknown status";
    }
}

const char* fs_kernel_name(int kernel) {
    switch (kernel) {
        case FS_KERNEL_AUTO: return "auto";
        case FS_KERNEL_WARP: return "warp";
        case FS_KERNEL_BLOCK: return "block";
        case FS_KERNEL_BLOCK_TMA: return "block_tma";
        case FS_KERNEL_CLUSTER: return "cluster";
        case FS_KERNEL_GENERIC: return "generic";
        default: return "unknown";
    }
}

const char* fs_version(void) {
#ifdef FS_DEBUG_BOUNDS
    return "libfsoftmax 0.2 (sm_100a, checked build)";
#else
    return "libfsoftmax 0.2 (sm_100a)";
#endif
}

}  // extern "C"
