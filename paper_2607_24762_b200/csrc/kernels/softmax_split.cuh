// Softmax of rows too long for a cluster's shared memory (more than 16 x 192 KiB): two kernels
// over a grid that fills the GPU, as for the normalisations.
//   sm_partial_kernel  block (row, b) reduces segment b of the row to one (reference, sum) pair,
//                      online over batches of four vectors per thread, and writes it to
//                      part[row * nseg + b]
//   sm_apply_kernel    the same grid: a block merges its row's nseg pairs (online-softmax merge),
//                      then writes y = 2^((x - R) c) / S for its segment, reading x again (from L2
//                      when the tensor fits) and taking the exponential a second time
// A negative scale is folded into the data (sign bits flipped on load, |scale| used), as in the
// log_softmax kernels. HBM traffic: one read and one write when x fits L2, else two reads.
#pragma once
#include "block_row.cuh"
#include "common.cuh"
#include "log_softmax.cuh"

namespace fsm {

template <int DT>
__global__ void __launch_bounds__(256)
sm_partial_kernel(const LsmParams p, float2* __restrict__ part, const int nseg, const int seg_vecs) {
    constexpr int NP = Traits<DT>::VE / 2;
    __shared__ float2 wp[32];
    pdl_launch_dependents();
    const int T = blockDim.x, tid = threadIdx.x;
    const int64_t row = blockIdx.x / nseg;
    const int b = static_cast<int>(blockIdx.x % nseg);
    const int64_t v0 = int64_t(b) * seg_vecs;
    const int nv = static_cast<int>(min(int64_t(seg_vecs), p.nvec - v0));
    const uint4* __restrict__ xv = static_cast<const uint4*>(p.x) + row * p.nvec + v0;
    const float ident = ref_identity<false>();
    const f32x2 c2 = pair(p.c, p.c);
    pdl_wait();
    float r = ident, s = 0.0f;
    for (int base = 0; base < nv; base += 4 * T) {
        uint4 raw[4];
        RefAcc<DT, false> ref;
        ref.init();
        const uint32_t idw = ident_word<DT, false>();
#pragma unroll
        for (int u = 0; u < 4; ++u) {
            raw[u] = make_uint4(idw, idw, idw, idw);                    // absent vectors drop out
            if (base + tid + u * T < nv) raw[u] = flip_vec(ld_keep(xv + base + tid + u * T), p.flip);
            ref.fold(raw[u]);
        }
        const float rc = ref.value();
        const float ru = (rc == ident) ? 0.0f : rc;
        const f32x2 ru2 = pair(ru, ru);
        f32x2 acc[2] = {pair(0.0f, 0.0f), pair(0.0f, 0.0f)};
#pragma unroll
        for (int u = 0; u < 4; ++u) {
            if (base + tid + u * T < nv) {                              // (a zero scale would make -inf * 0 of the padding NaN)
                f32x2 d[NP];
                lsm_accumulate<DT>(raw[u], ru2, c2, d, acc);
            }
        }
        const float partial = pair_sum(add2(acc[0], acc[1]));
        const float rn = fmaxf(r, rc);
        const bool keep = (rn == r);
        const float lo = keep ? rc : r;
        const float f = (lo == ident) ? 1.0f : ex2_ftz((lo - rn) * p.c);
        s = keep ? fmaf(partial, f, s) : fmaf(s, f, partial);
        r = rn;
    }
    block_merge_pairs<false>(r, s, wp, p.c);
    if (tid == 0) part[blockIdx.x] = make_float2(r, s);
}

template <int DT>
__global__ void __launch_bounds__(256)
sm_apply_kernel(const LsmParams p, const float2* __restrict__ part, const int nseg, const int seg_vecs) {
    constexpr int NP = Traits<DT>::VE / 2;
    pdl_launch_dependents();
    const int T = blockDim.x, tid = threadIdx.x, lane = tid & 31;
    const int64_t row = blockIdx.x / nseg;
    const int b = static_cast<int>(blockIdx.x % nseg);
    const int64_t v0 = int64_t(b) * seg_vecs;
    const int nv = static_cast<int>(min(int64_t(seg_vecs), p.nvec - v0));
    const uint4* __restrict__ xv = static_cast<const uint4*>(p.x) + row * p.nvec + v0;
    uint4* __restrict__ yv = static_cast<uint4*>(p.y) + row * p.nvec + v0;
    const float ident = ref_identity<false>();
    pdl_wait();
    // every warp merges the row's pairs: per lane online, then across the lanes
    float R = ident, S = 0.0f;
    for (int j = lane; j < nseg; j += 32) {
        const float2 v = part[row * nseg + j];
        const float rn = fmaxf(R, v.x);
        const float fa = ref_factor(R, rn, p.c, ident), fb = ref_factor(v.x, rn, p.c, ident);
        S = S * fa + v.y * fb;
        R = rn;
    }
    warp_merge_pairs<false>(R, S, p.c);
    // bf16 keeps its subnormal outputs: e carries 2^64, the reciprocal 2^-64 (see ex2_elem)
    const float bias = DT == DT_BF16 ? 64.0f : 0.0f;
    const float inv = recip<DT>(S) * (DT == DT_BF16 ? 0x1p-64f : 1.0f);
    const f32x2 R2 = pair(R, R), c2 = pair(p.c, p.c), b2 = pair(bias, bias), i2 = pair(inv, inv);
    for (int base = 0; base < nv; base += 4 * T) {
        uint4 raw[4];
#pragma unroll
        for (int u = 0; u < 4; ++u) {
            raw[u] = make_uint4(0u, 0u, 0u, 0u);
            if (base + tid + u * T < nv) raw[u] = flip_vec(ld_stream(xv + base + tid + u * T), p.flip);
        }
#pragma unroll
        for (int u = 0; u < 4; ++u) {
            if (base + tid + u * T < nv) {
                f32x2 d[NP];
                widen_pairs<DT>(raw[u], d);
#pragma unroll
                for (int k = 0; k < NP; ++k) {
                    float lo, hi;
                    unpair(fma2(sub2(d[k], R2), c2, b2), lo, hi);
                    d[k] = mul2(pair(ex2_ftz(lo), ex2_ftz(hi)), i2);
                }
                st_stream(yv + base + tid + u * T, narrow_pairs<DT>(d));
            }
        }
    }
}

}  // namespace fsm
