// Backward of y = softmax(scale * x):  dx_j = scale * y_j * (dy_j - sum_k dy_k y_k).
// Two inputs (dy, y), one output, one row-wide sum: the softmax skeleton with a plain dot product in
// place of the (max, sum) pair and no exponential. Algorithmic traffic: 3 elements per element.
//
//   smb_warp_kernel     (sub-)warp per row, both rows in registers (rows up to 4 KiB)
//   smb_tile_kernel     rows of 4-8 KiB: four rows per block in shared memory, a warp per row
//   smb_smem_kernel     row split over a cluster of 1..16 blocks; the dy and y slices are resident
//                       in shared memory (two bulk copies per chunk on one mbarrier), the partial
//                       dot products merge warp -> block -> cluster (st.async deposits), pass 2
//                       forms dx from the resident slices
//   smb_generic_kernel  block per row, element-wise, any shape and alignment
#pragma once
#include "common.cuh"
#include "norm_row.cuh"

namespace fsm {

struct SmbParams {
    const void* dy;
    const void* y;
    void* dx;
    int64_t rows;
    int64_t cols;
    int64_t nvec;
    float scale;
    int* status;
    int64_t pf_rows;
    float lag_ns;          // first wave of a one-shot grid: cluster i < lag_rows starts i * lag_ns late
    int lag_rows;
    int early_pf;          // first wave: ask L2 for the block's own input before griddepcontrol.wait (pdl_early_prefetch)
};

// ---------------------------------------------------------------------------------------------
template <int DT, int LANES, int VPL>
__global__ void __launch_bounds__(128)
smb_warp_kernel(const SmbParams p) {
    constexpr int NP = Traits<DT>::VE / 2;
    constexpr int G = 32 / LANES;
    pdl_launch_dependents();
    const int lane = threadIdx.x & 31;
    const int sub = lane / LANES, sl = lane % LANES;
    const int warps = blockDim.x >> 5;
    const int nvec = static_cast<int>(p.nvec);
    const uint4* __restrict__ gv = static_cast<const uint4*>(p.dy);
    const uint4* __restrict__ yv = static_cast<const uint4*>(p.y);
    uint4* __restrict__ dv = static_cast<uint4*>(p.dx);
    const f32x2 s2 = pair(p.scale, p.scale);
    pdl_wait();
    const int64_t ngroups = (p.rows + G - 1) / G;
    for (int64_t grp = int64_t(blockIdx.x) * warps + (threadIdx.x >> 5); grp < ngroups; grp += int64_t(gridDim.x) * warps) {
        const int64_t row = grp * G + sub;
        const bool row_ok = row < p.rows;
        uint4 graw[VPL], yraw[VPL];
#pragma unroll
        for (int k = 0; k < VPL; ++k) {
            graw[k] = make_uint4(0u, 0u, 0u, 0u); yraw[k] = make_uint4(0u, 0u, 0u, 0u);
            if (row_ok && sl + k * LANES < nvec) {
                graw[k] = ld_stream(gv + row * p.nvec + sl + k * LANES);
                yraw[k] = ld_stream(yv + row * p.nvec + sl + k * LANES);
            }
        }
        // the rows stay packed in registers and are widened where they are used (twice): two
        // widened rows of eight vectors per lane would not fit the register file
        f32x2 acc[2] = {pair(0.0f, 0.0f), pair(0.0f, 0.0f)};
#pragma unroll
        for (int k = 0; k < VPL; ++k) {
            f32x2 g[NP], y[NP];
            widen_pairs<DT>(graw[k], g);                    // absent vectors are zeros: they add nothing
            widen_pairs<DT>(yraw[k], y);
#pragma unroll
            for (int j = 0; j < NP; ++j) acc[j & 1] = fma2(g[j], y[j], acc[j & 1]);
        }
        const float dot = warp_sum<LANES>(pair_sum(add2(acc[0], acc[1])));
        const f32x2 d2 = pair(dot, dot);
        if (row_ok) {
#pragma unroll
            for (int k = 0; k < VPL; ++k) {
                if (sl + k * LANES < nvec) {
                    f32x2 g[NP], y[NP];
                    widen_pairs<DT>(graw[k], g);
                    widen_pairs<DT>(yraw[k], y);
#pragma unroll
                    for (int j = 0; j < NP; ++j) g[j] = mul2(mul2(y[j], sub2(g[j], d2)), s2);
                    st_stream(dv + row * p.nvec + sl + k * LANES, narrow_pairs<DT>(g));
                }
            }
        }
    }
}

// ---------------------------------------------------------------------------------------------
// Rows of 4-8 KiB: four rows per block; the dy row and the y row of a warp come to shared memory
// by two bulk copies on one mbarrier, and the warp works on them alone (dot product, then dx),
// with no block barrier after start-up. One-shot grid: block b handles rows b*W .. b*W+W-1.
// dynamic shared memory: W dy rows | W y rows | W mbarriers
// ---------------------------------------------------------------------------------------------
template <int DT>
__global__ void __launch_bounds__(128)
smb_tile_kernel(const SmbParams p) {
    constexpr int NP = Traits<DT>::VE / 2;
    constexpr int H = 4;                                   // vectors per lane and batch
    pdl_launch_dependents();
    extern __shared__ __align__(128) unsigned char smem[];
    const int lane = threadIdx.x & 31, w = threadIdx.x >> 5, W = blockDim.x >> 5;
    const int nvec = static_cast<int>(p.nvec);
    const uint32_t row_bytes = static_cast<uint32_t>(p.nvec) * 16u;          // at most 32 KiB: one copy each
    uint64_t* bars = reinterpret_cast<uint64_t*>(smem + 2 * size_t(W) * row_bytes);
    const int64_t row = int64_t(blockIdx.x) * W + w;
    if (threadIdx.x == 0) {
        for (int i = 0; i < W; ++i) mbar_init(smem_u32(&bars[i]), 1);
        mbar_fence_init();
        fence_proxy_async_smem();
    }
    __syncthreads();
    const char* gb = static_cast<const char*>(p.dy) + row * int64_t(row_bytes);
    const char* yb = static_cast<const char*>(p.y) + row * int64_t(row_bytes);
    pdl_wait();
    if (row >= p.rows) return;                             // no block-wide barrier follows
    if (lane == 0) {
        first_wave_lag(blockIdx.x, p.lag_ns, p.lag_rows);
        const uint32_t bar = smem_u32(&bars[w]);
        mbar_expect_tx(bar, 2u * row_bytes);
        bulk_load(smem_u32(smem) + uint32_t(w) * row_bytes, gb, row_bytes, bar);
        bulk_load(smem_u32(smem) + uint32_t(W + w) * row_bytes, yb, row_bytes, bar);
        if (p.pf_rows > 0 && row + p.pf_rows < p.rows) {
            l2_prefetch(gb + p.pf_rows * int64_t(row_bytes), row_bytes);
            l2_prefetch(yb + p.pf_rows * int64_t(row_bytes), row_bytes);
        }
    }
    const uint4* sg = reinterpret_cast<const uint4*>(smem + size_t(w) * row_bytes) + lane;
    const uint4* sy = reinterpret_cast<const uint4*>(smem + size_t(W + w) * row_bytes) + lane;
    uint4* __restrict__ dv = static_cast<uint4*>(p.dx) + row * p.nvec + lane;
    mbar_wait_warp(smem_u32(&bars[w]), 0u, p.status);      // on a timeout the status word is set and the row is garbage

    f32x2 acc[2] = {pair(0.0f, 0.0f), pair(0.0f, 0.0f)};
    for (int k0 = 0; k0 < nvec; k0 += 32 * H) {
        uint4 graw[H], yraw[H];
#pragma unroll
        for (int u = 0; u < H; ++u) {
            graw[u] = make_uint4(0u, 0u, 0u, 0u); yraw[u] = graw[u];          // absent vectors are zeros: they add nothing
            if (k0 + u * 32 + lane < nvec) { graw[u] = sg[k0 + u * 32]; yraw[u] = sy[k0 + u * 32]; }
        }
#pragma unroll
        for (int u = 0; u < H; ++u) {
            f32x2 g[NP], y[NP];
            widen_pairs<DT>(graw[u], g);
            widen_pairs<DT>(yraw[u], y);
#pragma unroll
            for (int j = 0; j < NP; ++j) acc[j & 1] = fma2(g[j], y[j], acc[j & 1]);
        }
    }
    const float dot = warp_sum<32>(pair_sum(add2(acc[0], acc[1])));
    const f32x2 d2 = pair(dot, dot), s2 = pair(p.scale, p.scale);
    for (int k0 = 0; k0 < nvec; k0 += 32 * H) {
        uint4 graw[H], yraw[H];
#pragma unroll
        for (int u = 0; u < H; ++u) {
            graw[u] = make_uint4(0u, 0u, 0u, 0u); yraw[u] = graw[u];
            if (k0 + u * 32 + lane < nvec) { graw[u] = sg[k0 + u * 32]; yraw[u] = sy[k0 + u * 32]; }
        }
#pragma unroll
        for (int u = 0; u < H; ++u) {
            if (k0 + u * 32 + lane < nvec) {
                f32x2 g[NP], y[NP];
                widen_pairs<DT>(graw[u], g);
                widen_pairs<DT>(yraw[u], y);
#pragma unroll
                for (int j = 0; j < NP; ++j) g[j] = mul2(mul2(y[j], sub2(g[j], d2)), s2);
                st_stream(dv + k0 + u * 32, narrow_pairs<DT>(g));
            }
        }
    }
}

// ---------------------------------------------------------------------------------------------
// cluster per row (one-shot grid). dynamic shared memory: dy slice | y slice (each stage_bytes,
// whole chunks) | 8 chunk mbarriers
// ---------------------------------------------------------------------------------------------
template <int DT, bool FULL>
__global__ void __launch_bounds__(256, 3)
smb_smem_kernel(const SmbParams p, const uint32_t stage_bytes, const int slice, const int nchunk_full) {
    constexpr int VE = Traits<DT>::VE;
    constexpr int NP = VE / 2;
    constexpr int U = 8;
    pdl_launch_dependents();
    extern __shared__ __align__(128) unsigned char smem[];
    __shared__ float wp[32];
    __shared__ __align__(16) float2 xchg[16];
    __shared__ __align__(8) uint64_t xbar;
    const int T = blockDim.x, tid = threadIdx.x, lane = tid & 31, nwarps = T >> 5;
    const int tpos = (tid >> 5) * (32 * U) + lane;
    const uint32_t q = cluster_ctarank(), cs = cluster_nctarank();
    const int64_t row = cluster_id_x();
    const int chunk_vecs = U * T;
    int v0, nv, nchunk;
    if (FULL) {
        v0 = static_cast<int>(q) * slice; nv = slice; nchunk = nchunk_full;
    } else {
        const int nvec = static_cast<int>(p.nvec);
        v0 = min(nvec, static_cast<int>(q) * slice);
        nv = min(nvec, v0 + slice) - v0;
        nchunk = (nv + chunk_vecs - 1) / chunk_vecs;
    }
    uint64_t* bars = reinterpret_cast<uint64_t*>(smem + 2 * size_t(stage_bytes));
    const uint4* sg = reinterpret_cast<const uint4*>(smem) + tpos;
    const uint4* sy = reinterpret_cast<const uint4*>(smem + stage_bytes) + tpos;
    const int64_t row_bytes = p.nvec * 16;
    const char* gb = static_cast<const char*>(p.dy) + int64_t(v0) * 16;
    const char* yb = static_cast<const char*>(p.y) + int64_t(v0) * 16;

    if (tid == 0) {
        for (int ch = 0; ch < kNormMaxChunks; ++ch) mbar_init(smem_u32(&bars[ch]), 1);
        mbar_init(smem_u32(&xbar), 1);
        mbar_fence_init();
        fence_proxy_async_smem();
        pdl_wait_first_wave<true>(row, p.lag_ns, p.lag_rows, p.early_pf, [&] { if (nv > 0) { pdl_early_prefetch(gb + row * row_bytes, int64_t(nv) * 16); pdl_early_prefetch(yb + row * row_bytes, int64_t(nv) * 16); } });
        for (int ch = 0; ch < nchunk; ++ch) {
            const uint32_t cv = uint32_t(FULL ? chunk_vecs : min(chunk_vecs, nv - ch * chunk_vecs)) * 16u;
            const uint32_t off = uint32_t(ch) * uint32_t(chunk_vecs) * 16u;
            const uint32_t bar = smem_u32(&bars[ch]);
            // both slices' pieces of the chunk complete the same barrier (cv <= 32 KiB: one copy each)
            mbar_expect_tx(bar, 2u * cv);
            bulk_load(smem_u32(smem) + off, gb + row * row_bytes + off, cv, bar);
            bulk_load(smem_u32(smem) + stage_bytes + off, yb + row * row_bytes + off, cv, bar);
        }
        if (p.pf_rows > 0 && row + p.pf_rows < p.rows && nv > 0) {
            l2_prefetch(gb + (row + p.pf_rows) * row_bytes, uint32_t(nv) * 16u);
            l2_prefetch(yb + (row + p.pf_rows) * row_bytes, uint32_t(nv) * 16u);
        }
        if (cs > 1) mbar_expect_tx(smem_u32(&xbar), cs * 8u);
    }
    __syncthreads();
    if (cs > 1) {
        cluster_arrive_relaxed();
        cluster_wait_acquire();
    }
    pdl_wait();

    // ---- pass 1: the dot product over the chunks as they land
    bool alive = true;
    f32x2 acc[2] = {pair(0.0f, 0.0f), pair(0.0f, 0.0f)};
    for (int ch = 0; ch < nchunk; ++ch) {
        if (tid < 32 && alive) alive = mbar_wait_warp(smem_u32(&bars[ch]), 0u, p.status);
        if (T > 32) __syncthreads();
        const int off = ch * chunk_vecs;
        const int cbase = off + tpos;
#pragma unroll
        for (int h = 0; h < 2; ++h) {
            uint4 graw[U / 2], yraw[U / 2];
#pragma unroll
            for (int u = 0; u < U / 2; ++u) {
                const int uu = h * (U / 2) + u;
                graw[u] = sg[off + uu * 32]; yraw[u] = sy[off + uu * 32];
                if (!FULL && cbase + uu * 32 >= nv) { graw[u] = make_uint4(0u, 0u, 0u, 0u); yraw[u] = make_uint4(0u, 0u, 0u, 0u); }
            }
#pragma unroll
            for (int u = 0; u < U / 2; ++u) {
                f32x2 g[NP], y[NP];
                widen_pairs<DT>(graw[u], g);
                widen_pairs<DT>(yraw[u], y);
#pragma unroll
                for (int k = 0; k < NP; ++k) acc[k & 1] = fma2(g[k], y[k], acc[k & 1]);
            }
        }
    }
    float dot = warp_sum<32>(pair_sum(add2(acc[0], acc[1])));
    if (nwarps > 1) {
        if (lane == 0) wp[tid >> 5] = dot;
        __syncthreads();
        dot = warp_sum<32>(lane < nwarps ? wp[lane] : 0.0f);
    }
    if (cs > 1) {
        if (tid < cs) st_async_v2(map_to_rank(smem_u32(&xchg[q]), tid), dot, 0.0f, map_to_rank(smem_u32(&xbar), tid));
        cluster_arrive_relaxed();          // exit guard: waited for after pass 2 (see smem_row.cuh)
        if (tid < 32 && alive) alive = mbar_wait_warp(smem_u32(&xbar), 0u, p.status);
        if (T > 32) __syncthreads();
        float a = 0.0f, b = 0.0f;
        if (lane < static_cast<int>(cs)) ld_shared_v2(smem_u32(&xchg[lane]), a, b);
        dot = warp_sum<32>(a);
    }

    // ---- pass 2: dx = scale * y * (dy - dot) from the resident slices
    const f32x2 d2 = pair(dot, dot), s2 = pair(p.scale, p.scale);
    uint4* __restrict__ dv = static_cast<uint4*>(p.dx) + row * p.nvec + v0 + tpos;
    for (int ch = 0; ch < nchunk; ++ch) {
        const int off = ch * chunk_vecs;
        const int cbase = off + tpos;
#pragma unroll
        for (int h = 0; h < 2; ++h) {
            uint4 graw[U / 2], yraw[U / 2];
#pragma unroll
            for (int u = 0; u < U / 2; ++u) { graw[u] = sg[off + (h * (U / 2) + u) * 32]; yraw[u] = sy[off + (h * (U / 2) + u) * 32]; }
#pragma unroll
            for (int u = 0; u < U / 2; ++u) {
                const int uu = h * (U / 2) + u;
                if (FULL || cbase + uu * 32 < nv) {
                    f32x2 g[NP], y[NP];
                    widen_pairs<DT>(graw[u], g);
                    widen_pairs<DT>(yraw[u], y);
#pragma unroll
                    for (int k = 0; k < NP; ++k) g[k] = mul2(mul2(y[k], sub2(g[k], d2)), s2);
                    st_stream(dv + off + uu * 32, narrow_pairs<DT>(g));
                }
            }
        }
    }
    if (cs > 1) cluster_wait_acquire();    // no block leaves while a peer's deposit into it is still to be issued
}

// ---------------------------------------------------------------------------------------------
template <int DT>
__global__ void __launch_bounds__(1024)
smb_generic_kernel(const SmbParams p) {
    __shared__ float red[32];
    pdl_launch_dependents();
    pdl_wait();
    for (int64_t row = blockIdx.x; row < p.rows; row += gridDim.x) {
        const int64_t base = row * p.cols;
        float s = 0.0f;
        for (int64_t j = threadIdx.x; j < p.cols; j += blockDim.x)
            s = fmaf(load_elem<DT>(p.dy, base + j), load_elem<DT>(p.y, base + j), s);
        const float dot = block_sum(s, red);
        for (int64_t j = threadIdx.x; j < p.cols; j += blockDim.x)
            store_elem<DT>(p.dx, base + j, load_elem<DT>(p.y, base + j) * (load_elem<DT>(p.dy, base + j) - dot) * p.scale);
    }
}

}  // namespace fsm
