// (Sub-)warp-per-row softmax, the row held in registers (short rows: MoE-router-sized up to a few KB).
//
// LANES consecutive lanes own one row, a warp covers G = 32/LANES adjacent rows per pass, and R
// passes are unrolled so that all R*VPL 16-byte loads of a lane are in flight before any
// arithmetic. Lane l of a row's group reads vectors l, l+LANES, ...: every warp-wide load or
// store covers whole 32-byte sectors of G adjacent rows. The row maximum and sum are warp-shuffle
// reductions over the group; one ex2 per element.
//
// warp_row_kernel takes its rows by 128-bit global loads straight into registers. (A variant that
// brought a block's tile of consecutive rows into shared memory with one bulk copy was measured
// slower on every short-row shape and is gone.) softmax_tile_kernel, at the end of this file,
// serves the 16-bit rows a warp can no longer hold in registers: one warp per row from shared memory.
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
    if (LANES * VPL >= 128 && p.early_pf && lane == 0) {
        // rows of 2 KiB and more: this warp's first tile (contiguous rows) is asked of L2 ahead of the
        // dependency wait (pdl_early_prefetch); measured 21.77 -> 21.57 us on 16384 rows of 4 KiB bf16,
        // while 256-byte rows lose (12.02 -> 12.09 us on 131072 of them) and go without
        const int64_t tile0 = int64_t(blockIdx.x) * warps + (threadIdx.x >> 5);
        if (tile0 < ntiles) {
            const int64_t r0 = tile0 * rows_per_tile;
            pdl_early_prefetch(reinterpret_cast<const char*>(xv + r0 * p.nvec), min(rows_per_tile, p.rows - r0) * p.nvec * 16);
        }
    }
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

// ---------------------------------------------------------------------------------------------
// 16-bit rows of 4-12 KiB: four rows per block, each brought to shared memory by a bulk copy of its
// own (one mbarrier per row) and worked on by one warp alone, three reads of shared memory:
//   pass A  the row reference R (packed max over the raw vectors, one shuffle reduction);
//   pass B  e = 2^((x - R) c): subtraction first (exact), one ex2 per element, the row sum taken over
//           the unrounded fp32 values, e written back IN PLACE in the element dtype (only the lane
//           that wrote a vector reads it again);
//   pass C  y = e / S, 128-bit streaming stores.
// No block barrier after start-up and a register footprint that does not grow with the row, so
// six to nine blocks of four warps stay resident per SM: the rows a (sub-)warp can no longer hold in
// registers and a cluster's chunked slices serve poorly. Storing e rounded to the element dtype
// keeps the result within one unit in the last place of the correctly rounded value (the argument
// in smem_row.cuh). One-shot grid: block b handles rows b*W .. b*W+W-1.
// dynamic shared memory: W rows | W mbarriers
// ---------------------------------------------------------------------------------------------
template <int DT, bool NEG>
__global__ void __launch_bounds__(128)
softmax_tile_kernel(const Params p) {
    static_assert(DT != DT_F32, "16-bit element types only");
    constexpr int VE = Traits<DT>::VE;
    constexpr int H = 4;                                   // vectors per lane and batch
    pdl_launch_dependents();
    extern __shared__ __align__(128) unsigned char smem[];
    const int lane = threadIdx.x & 31, w = threadIdx.x >> 5, W = blockDim.x >> 5;
    const int nvec = static_cast<int>(p.nvec);
    const int64_t row_bytes = p.nvec * 16;
    uint64_t* bars = reinterpret_cast<uint64_t*>(smem + size_t(W) * size_t(row_bytes));
    const int64_t row = int64_t(blockIdx.x) * W + w;
    if (threadIdx.x == 0) {
        for (int i = 0; i < W; ++i) mbar_init(smem_u32(&bars[i]), 1);
        mbar_fence_init();
        fence_proxy_async_smem();
    }
    __syncthreads();
    const char* xb = static_cast<const char*>(p.x);
    pdl_wait();
    if (row >= p.rows) return;                             // no block-wide barrier follows
    if (lane == 0) {
        first_wave_lag(blockIdx.x, p.lag_ns, p.lag_rows);
        bulk_load_row(smem_u32(smem) + uint32_t(w) * uint32_t(row_bytes), xb + row * row_bytes, uint32_t(row_bytes), smem_u32(&bars[w]));
        if (p.pf_rows > 0 && row + p.pf_rows < p.rows) l2_prefetch(xb + (row + p.pf_rows) * row_bytes, uint32_t(row_bytes));
    }
    uint4* sv = reinterpret_cast<uint4*>(smem + size_t(w) * size_t(row_bytes)) + lane;
    uint4* __restrict__ yv = static_cast<uint4*>(p.y) + row * p.nvec + lane;
    const float ident = ref_identity<NEG>();
    mbar_wait_warp(smem_u32(&bars[w]), 0u, p.status);      // on a timeout the status word is set and the row is garbage

    RefAcc<DT, NEG> ref;
    ref.init();
    for (int k0 = 0; k0 < nvec; k0 += 32 * H) {
#pragma unroll
        for (int u = 0; u < H; ++u)
            if (k0 + u * 32 + lane < nvec) ref.fold(sv[k0 + u * 32]);
    }
    const float R = warp_pick<32, NEG>(ref.value());
    // a row whose reference is still the identity (only masked entries) subtracts 0 instead: -inf - 0 stays
    // -inf, the sum is 0 and 0 * (1 / 0) makes the row NaN, as the formula does
    const float ru = (R == ident) ? 0.0f : R;
    const f32x2 r2 = pair(ru, ru), c2 = pair(p.c, p.c);
    f32x2 acc[VE / 2];
#pragma unroll
    for (int k = 0; k < VE / 2; ++k) acc[k] = pair(0.0f, 0.0f);
    for (int k0 = 0; k0 < nvec; k0 += 32 * H) {
        uint4 raw[H];
#pragma unroll
        for (int u = 0; u < H; ++u)
            if (k0 + u * 32 + lane < nvec) raw[u] = sv[k0 + u * 32];
#pragma unroll
        for (int u = 0; u < H; ++u)
            if (k0 + u * 32 + lane < nvec) sv[k0 + u * 32] = ex2_vec<DT>(raw[u], r2, c2, acc);
    }
#pragma unroll
    for (int k = 1; k < VE / 2; ++k) acc[0] = add2(acc[0], acc[k]);
    const float inv = recip<DT>(warp_sum<32>(pair_sum(acc[0])));
    const f32x2 i2 = pair(inv, inv);
    for (int k0 = 0; k0 < nvec; k0 += 32 * H) {
        uint4 e[H];
#pragma unroll
        for (int u = 0; u < H; ++u)
            if (k0 + u * 32 + lane < nvec) e[u] = sv[k0 + u * 32];
#pragma unroll
        for (int u = 0; u < H; ++u)
            if (k0 + u * 32 + lane < nvec) st_stream(yv + k0 + u * 32, scale_vec<DT, false>(e[u], i2, i2));
    }
}

}  // namespace fsm
