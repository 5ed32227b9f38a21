// Router step of a mixture-of-experts layer on warp-resident rows: softmax over the expert
// logits, then the k largest probabilities (ties to the lower column), optionally renormalised
// over the selected ones. One (sub-)warp group of LANES lanes owns a row, as in warp_row_kernel;
// a lane holds VPL vectors, at most 32 elements.
//
// The order of the probabilities is the order of z = scale * x, so the selection is made on the
// inputs themselves, exactly: each element becomes an order-preserving 32-bit unsigned key
// (negated first when the scale is negative, all finite values equal when it is zero, NaN counted
// as -inf), 0 marks an element already taken. The keys live in shared memory, one column of
// NE words per thread (bank = thread: conflict-free whatever element a thread touches), so that
// a round touches only what it must: each lane keeps the maximum of each of its vectors in
// registers; a round takes the group maximum with a shuffle butterfly, lets the lanes that hold it
// find their lowest such column (8 shared loads), takes the lowest column with a second
// butterfly, and the owner clears that key and refreshes that one vector's maximum.
// The weight of a selected element is 2^((key - key_0)|c|) over the row sum (or over the sum of
// the selected ones), which needs no access to the element itself.
#pragma once
#include "common.cuh"

namespace fsm {

struct RouterParams {
    const void* x;
    float* w;          // [rows, k] weights, selection order
    int* idx;          // [rows, k] columns, selection order
    int64_t rows;
    int64_t nvec;      // 16-byte vectors per row
    int k;
    float c;           // scale * log2(e)
    int renorm;
};

__device__ __forceinline__ uint32_t order_key(float v) {        // monotone float -> uint32, all results >= 1
    const uint32_t b = __float_as_uint(v);
    return (b & 0x80000000u) ? ~b : (b | 0x80000000u);
}
__device__ __forceinline__ float order_unkey(uint32_t u) {
    return __uint_as_float((u & 0x80000000u) ? (u & 0x7fffffffu) : ~u);
}

__device__ __forceinline__ float ex2_ftz_r(float t) {
    float r;
    asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(r) : "f"(t));
    return r;
}

// Dynamic shared memory: NE * blockDim.x 32-bit keys, element-major ([element][thread]).
template <int DT, int LANES, int VPL>
__global__ void __launch_bounds__(128)
router_topk_kernel(const RouterParams p) {
    constexpr int VE = Traits<DT>::VE;
    constexpr int G = 32 / LANES;
    pdl_launch_dependents();
    extern __shared__ uint32_t keys[];
    const int T = blockDim.x, tid = threadIdx.x;
    const int lane = tid & 31;
    const int sub = lane / LANES, sl = lane % LANES;
    const int warps = T >> 5;
    const int nvec = static_cast<int>(p.nvec);
    const uint4* __restrict__ xv = static_cast<const uint4*>(p.x);
    const float cabs = fabsf(p.c);
    const float sg = p.c > 0.0f ? 1.0f : (p.c < 0.0f ? -1.0f : 0.0f);   // z-order: x, -x, or all finite values equal
    uint32_t* kt = keys + tid;                                          // this thread's column
    pdl_wait();

    const int64_t ngroups = (p.rows + G - 1) / G;
    for (int64_t grp = int64_t(blockIdx.x) * warps + (tid >> 5); grp < ngroups; grp += int64_t(gridDim.x) * warps) {
        const int64_t row = grp * G + sub;
        const bool row_ok = row < p.rows;
        // ---- load; z-ordered values; row maximum
        float z[VPL][VE];
        bool live[VPL];
        float top = __int_as_float(0xff800000);
#pragma unroll
        for (int v = 0; v < VPL; ++v) {
            live[v] = row_ok && sl + v * LANES < nvec;
            uint4 raw = make_uint4(0u, 0u, 0u, 0u);
            if (live[v]) raw = ld_stream(xv + row * p.nvec + sl + v * LANES);
            unpack<DT>(raw, z[v]);
#pragma unroll
            for (int i = 0; i < VE; ++i) {
                z[v][i] = fmaf(z[v][i], sg, 0.0f);          // sign of the scale; -0 becomes +0; inf * 0 = NaN
                if (live[v]) top = fmaxf(top, z[v][i]);     // fmaxf drops NaN
            }
        }
        top = warp_pick<LANES, false>(top);
        // ---- row sum (a NaN or +inf value, or a row of -inf only, makes it NaN); keys to shared memory
        float s = 0.0f;
        uint32_t m[VPL];
#pragma unroll
        for (int v = 0; v < VPL; ++v) {
            m[v] = 0u;
#pragma unroll
            for (int i = 0; i < VE; ++i) {
                const float zz = z[v][i];
                if (live[v]) s += ex2_ftz_r((zz - top) * cabs);
                const float kz = (zz != zz) ? __int_as_float(0xff800000) : zz;   // NaN counts as -inf
                const uint32_t ku = live[v] ? order_key(kz) : 0u;                  // padding is never selected
                kt[(v * VE + i) * T] = ku;
                m[v] = max(m[v], ku);
            }
        }
        s = warp_sum<LANES>(s);
        const float inv_s = 1.0f / s;                              // NaN when the row is NaN
        float sel = 0.0f;
        float key0 = 0.0f;
        for (int r = 0; r < p.k; ++r) {
            uint32_t lb = m[0];
#pragma unroll
            for (int v = 1; v < VPL; ++v) lb = max(lb, m[v]);
            uint32_t M = lb;                                        // the group's best remaining key
#pragma unroll
            for (int o = LANES / 2; o > 0; o >>= 1) M = max(M, __shfl_xor_sync(0xffffffffu, M, o));
            int mycol = 0x7fffffff, vv = 0, ii = 0;
            uint32_t rest = 0u;                                     // maximum of that vector without the taken element
            if (lb == M && M != 0u) {                               // this lane holds it: its lowest such column
#pragma unroll
                for (int v = VPL - 1; v >= 0; --v) if (m[v] == M) vv = v;
                bool found = false;
#pragma unroll
                for (int i = 0; i < VE; ++i) {
                    const uint32_t kv = kt[(vv * VE + i) * T];
                    const bool hit = !found && kv == M;
                    if (hit) ii = i;
                    found = found || hit;
                    rest = max(rest, hit ? 0u : kv);
                }
                mycol = (vv * LANES + sl) * VE + ii;
            }
            int col = mycol;                                        // equal keys: the lowest column wins
#pragma unroll
            for (int o = LANES / 2; o > 0; o >>= 1) col = min(col, __shfl_xor_sync(0xffffffffu, col, o));
            if (mycol == col && col != 0x7fffffff) {                // owner: take it out, refresh that vector's maximum
                kt[(vv * VE + ii) * T] = 0u;
#pragma unroll
                for (int v = 0; v < VPL; ++v) if (v == vv) m[v] = rest;
            }
            const float kf = order_unkey(M);
            if (r == 0) key0 = kf;
            const float e = ex2_ftz_r((kf - key0) * cabs);
            sel += e;
            if (row_ok && sl == 0) {
                p.idx[row * p.k + r] = col;
                p.w[row * p.k + r] = p.renorm ? e : e * inv_s;
            }
        }
        if (p.renorm && row_ok && sl == 0) {
            // 0 * inv_s carries a NaN row into the renormalised weights (inv_s is finite otherwise)
            const float f = 1.0f / sel + 0.0f * inv_s;
            for (int r = 0; r < p.k; ++r) p.w[row * p.k + r] *= f;
        }
    }
}

}  // namespace fsm
