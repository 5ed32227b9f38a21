// (Sub-)warp-per-row softmax, the row held in registers (short rows: MoE-router-sized up to a few KB).
//
// LANES consecutive lanes own one row, a warp covers G = 32/LANES adjacent rows per pass, and R
// passes are unrolled so that all R*VPL 16-byte loads of a lane are in flight before any
// arithmetic. Lane l of a row's group reads vectors l, l+LANES, ...: every warp-wide load or
// store covers G*LANES*16 contiguous bytes. The row maximum and sum are warp-shuffle reductions
// over the group; one ex2 per element.
#pragma once
#include "common.cuh"

namespace fsm {

template <int DT, int LANES, int VPL, int R>
__global__ void __launch_bounds__(256)
warp_row_kernel(const Params p) {
    constexpr int VE = Traits<DT>::VE;
    constexpr int G = 32 / LANES;
    const int lane = threadIdx.x & 31;
    const int sub = lane / LANES;          // which of the warp's G rows
    const int sl = lane % LANES;           // lane within the row's group
    const int warps = blockDim.x >> 5;
    const int64_t rows_per_tile = int64_t(G) * R;
    const int64_t ntiles = (p.rows + rows_per_tile - 1) / rows_per_tile;
    const float ident = ref_identity(p.neg);
    const uint4* __restrict__ xv = static_cast<const uint4*>(p.x);
    uint4* __restrict__ yv = static_cast<uint4*>(p.y);
    const int nvec = static_cast<int>(p.nvec);

    for (int64_t tile = int64_t(blockIdx.x) * warps + (threadIdx.x >> 5); tile < ntiles;
         tile += int64_t(gridDim.x) * warps) {
        uint4 raw[R][VPL];
        const int64_t row0 = tile * rows_per_tile + sub;
#pragma unroll
        for (int r = 0; r < R; ++r) {
            const int64_t row = row0 + int64_t(r) * G;
#pragma unroll
            for (int k = 0; k < VPL; ++k) {
                const int v = sl + k * LANES;
                raw[r][k] = make_uint4(0u, 0u, 0u, 0u);
                if (row < p.rows && v < nvec) raw[r][k] = ld_stream(xv + row * p.nvec + v);
            }
        }
#pragma unroll
        for (int r = 0; r < R; ++r) {
            const int64_t row = row0 + int64_t(r) * G;
            float e[VPL][VE];
            float ref = ident;
#pragma unroll
            for (int k = 0; k < VPL; ++k) {
                unpack<DT>(raw[r][k], e[k]);
                if (sl + k * LANES < nvec) {
#pragma unroll
                    for (int i = 0; i < VE; ++i) ref = ref_pick(ref, e[k][i], p.neg);
                }
            }
            ref = warp_pick<LANES>(ref, p.neg);
            float s = 0.0f;
#pragma unroll
            for (int k = 0; k < VPL; ++k) {
                if (sl + k * LANES < nvec) {
#pragma unroll
                    for (int i = 0; i < VE; ++i) {
                        e[k][i] = ex2<DT>((e[k][i] - ref) * p.c);
                        s += e[k][i];
                    }
                }
            }
            s = warp_sum<LANES>(s);
            const float inv = 1.0f / s;
            if (row < p.rows) {
#pragma unroll
                for (int k = 0; k < VPL; ++k) {
                    const int v = sl + k * LANES;
                    if (v < nvec) {
#pragma unroll
                        for (int i = 0; i < VE; ++i) e[k][i] *= inv;
                        st_stream(yv + row * p.nvec + v, pack<DT>(e[k]));
                    }
                }
            }
        }
    }
}

}  // namespace fsm
