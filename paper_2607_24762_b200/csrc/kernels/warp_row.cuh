// (Sub-)warp-per-row softmax, the row held in registers (short rows: MoE-router-sized up to a few KB).
//
// LANES consecutive lanes own one row, a warp covers G = 32/LANES adjacent rows per pass, and R
// passes are unrolled so that all R*VPL 16-byte loads of a lane are in flight before any
// arithmetic. Lane l of a row's group reads vectors l, l+LANES, ...: every warp-wide load or
// store covers whole 32-byte sectors of G adjacent rows. The row maximum and sum are warp-shuffle
// reductions over the group; one ex2 per element.
//
// Two front ends:
//   warp_row_kernel      128-bit global loads straight into registers
//   warp_row_tma_kernel  the block's tile of consecutive rows (one contiguous byte range) is
//                        brought into shared memory by one bulk async copy (no multicast) and the
//                        warps read their rows from there
#pragma once
#include "common.cuh"

namespace fsm {

// One row group's arithmetic, from raw vectors to stored output.
// fetch(k) returns the lane's k-th raw vector; live(k) says whether it exists.
template <int DT, bool NEG, int LANES, int VPL, typename Live>
__device__ __forceinline__ void warp_row_math(const uint4 (&raw)[VPL], float c, uint4* __restrict__ yrow,
                                              bool store, Live live) {
    constexpr int VE = Traits<DT>::VE;
    RefAcc<DT, NEG> acc;
    acc.init();
#pragma unroll
    for (int k = 0; k < VPL; ++k)
        if (live(k)) acc.fold(raw[k]);
    const float ref = warp_pick<LANES, NEG>(acc.value());
    float e[VPL][VE];
    float s = 0.0f;
#pragma unroll
    for (int k = 0; k < VPL; ++k) {
        unpack<DT>(raw[k], e[k]);
        if (live(k)) {
#pragma unroll
            for (int i = 0; i < VE; ++i) {
                e[k][i] = ex2_elem<DT>(e[k][i] - ref, c);
                s += e[k][i];
            }
        }
    }
    s = warp_sum<LANES>(s);
    const float inv = recip<DT>(s);
    if (store) {
#pragma unroll
        for (int k = 0; k < VPL; ++k) {
            if (live(k)) {
#pragma unroll
                for (int i = 0; i < VE; ++i) e[k][i] *= inv;
                st_stream(yrow + k * LANES, pack<DT>(e[k]));
            }
        }
    }
}

// Rows that fill 64 payload registers per lane are capped at 85 registers (3 blocks of 256
// threads per SM) so that enough rows are in flight to cover HBM latency.
template <int DT, int VPL, int R> struct WarpCfg {
    static constexpr int MIN_BLOCKS = (VPL * R * Traits<DT>::VE >= 64) ? 3 : 1;
};

template <int DT, bool NEG, int LANES, int VPL, int R>
__global__ void __launch_bounds__(256, WarpCfg<DT, VPL, R>::MIN_BLOCKS)
warp_row_kernel(const Params p) {
    constexpr int G = 32 / LANES;
    pdl_launch_dependents();
    const int lane = threadIdx.x & 31;
    const int sub = lane / LANES;          // which of the warp's G rows
    const int sl = lane % LANES;           // lane within the row's group
    const int warps = blockDim.x >> 5;
    const int64_t rows_per_tile = int64_t(G) * R;
    const int64_t ntiles = (p.rows + rows_per_tile - 1) / rows_per_tile;
    const uint4* __restrict__ xv = static_cast<const uint4*>(p.x);
    uint4* __restrict__ yv = static_cast<uint4*>(p.y);
    const int nvec = static_cast<int>(p.nvec);
    auto live = [&](int k) { return sl + k * LANES < nvec; };
    pdl_wait();

    for (int64_t tile = int64_t(blockIdx.x) * warps + (threadIdx.x >> 5); tile < ntiles;
         tile += int64_t(gridDim.x) * warps) {
        uint4 raw[R][VPL];
        const int64_t row0 = tile * rows_per_tile + sub;
        const int64_t off0 = row0 * p.nvec + sl;
#pragma unroll
        for (int r = 0; r < R; ++r) {
            const bool row_ok = row0 + int64_t(r) * G < p.rows;
            const uint4* xr = xv + off0 + int64_t(r) * G * p.nvec;
#pragma unroll
            for (int k = 0; k < VPL; ++k) {
                raw[r][k] = make_uint4(0u, 0u, 0u, 0u);
                if (row_ok && live(k)) raw[r][k] = ld_stream(xr + k * LANES);
            }
        }
#pragma unroll
        for (int r = 0; r < R; ++r) {
            const bool row_ok = row0 + int64_t(r) * G < p.rows;
            warp_row_math<DT, NEG, LANES, VPL>(raw[r], p.c, yv + off0 + int64_t(r) * G * p.nvec, row_ok, live);
        }
    }
}

// Dynamic shared memory: the tile (tile_rows * row bytes) followed by one mbarrier.
// The block's warps split the tile's rows G at a time; a block handles tiles
// blockIdx.x, blockIdx.x + gridDim.x, ... (normally exactly one).
template <int DT, bool NEG, int LANES, int VPL>
__global__ void __launch_bounds__(256)
warp_row_tma_kernel(const Params p, const int tile_rows, const uint32_t tile_bytes_max) {
    constexpr int G = 32 / LANES;
    pdl_launch_dependents();
    extern __shared__ __align__(128) unsigned char smem[];
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    const int sub = lane / LANES, sl = lane % LANES;
    const int warps = blockDim.x >> 5;
    const int nvec = static_cast<int>(p.nvec);
    const int64_t row_bytes = p.nvec * 16;
    const int64_t ntiles = (p.rows + tile_rows - 1) / tile_rows;
    uint64_t* bar = reinterpret_cast<uint64_t*>(smem + tile_bytes_max);
    const char* xb = static_cast<const char*>(p.x);
    uint4* __restrict__ yv = static_cast<uint4*>(p.y);
    auto live = [&](int k) { return sl + k * LANES < nvec; };

    if (threadIdx.x == 0) {
        mbar_init(smem_u32(bar), 1);
        mbar_fence_init();
        fence_proxy_async_smem();
    }
    __syncthreads();
    pdl_wait();
    uint32_t phase = 0;
    bool alive = true;
    for (int64_t tile = blockIdx.x; tile < ntiles; tile += gridDim.x) {
        const int64_t row_first = tile * tile_rows;
        const int nrows = static_cast<int>(min(int64_t(tile_rows), p.rows - row_first));
        if (threadIdx.x == 0)
            bulk_load_row(smem_u32(smem), xb + row_first * row_bytes, static_cast<uint32_t>(nrows * row_bytes), smem_u32(bar));
        if (alive) alive = mbar_wait_warp(smem_u32(bar), phase, p.status);
        phase ^= 1u;
        const uint4* tile_v = reinterpret_cast<const uint4*>(smem);
        for (int lr = warp * G + sub; lr - sub < nrows; lr += warps * G) {
            const bool row_ok = lr < nrows;
            uint4 raw[VPL];
#pragma unroll
            for (int k = 0; k < VPL; ++k) {
                raw[k] = make_uint4(0u, 0u, 0u, 0u);
                if (row_ok && live(k)) raw[k] = tile_v[int64_t(lr) * nvec + sl + k * LANES];
            }
            warp_row_math<DT, NEG, LANES, VPL>(raw, p.c, yv + (row_first + lr) * p.nvec + sl, row_ok, live);
        }
        if (tile + gridDim.x < ntiles) {   // another tile follows: everyone is done reading this one
            __syncthreads();
            if (threadIdx.x == 0) fence_proxy_async_smem();
        }
    }
}

}  // namespace fsm
