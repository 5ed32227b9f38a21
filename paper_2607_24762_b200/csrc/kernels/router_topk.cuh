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
// That kernel serves any k; router_top8_kernel below (k <= 8) selects with sorting networks in
// registers instead.
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
    int wide;          // k == 8 and w, idx 32-byte aligned: a row's eight weights (columns) leave in one 256-bit store
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

// ---------------------------------------------------------------------------------------------
// k <= 8: selection by sorting networks in registers, no shared memory and no rounds.
// An element becomes ONE integer key: the order-preserving image of its value in the high half,
// the complement of its column in the low half (16 + 16 bits for bf16/fp16 inputs, 32 + 32 for
// fp32), so that a plain integer maximum picks the larger value and, among equal values, the
// lower column; 0 marks padding. A lane sorts its elements in groups of eight (19
// compare-exchanges each) and merges the groups into its own eight best; two sorted lists merge
// into the eight best of both by c_i = max(a_i, b_{7-i}) (a bitonic sequence) and a 12-exchange
// bitonic sort. The lanes of a row merge their lists the same way through shuffles (both partners
// end with the same list), and lane r mod LANES writes entry r.
// ---------------------------------------------------------------------------------------------
template <class K> __device__ __forceinline__ void cmpx(K& a, K& b) {       // a >= b afterwards
    const K hi = max(a, b), lo = min(a, b);
    a = hi; b = lo;
}
template <class K> __device__ __forceinline__ void sort8_desc(K (&a)[8]) {
    cmpx(a[0], a[1]); cmpx(a[2], a[3]); cmpx(a[4], a[5]); cmpx(a[6], a[7]);
    cmpx(a[0], a[2]); cmpx(a[1], a[3]); cmpx(a[4], a[6]); cmpx(a[5], a[7]);
    cmpx(a[1], a[2]); cmpx(a[5], a[6]);
    cmpx(a[0], a[4]); cmpx(a[1], a[5]); cmpx(a[2], a[6]); cmpx(a[3], a[7]);
    cmpx(a[2], a[4]); cmpx(a[3], a[5]);
    cmpx(a[1], a[2]); cmpx(a[3], a[4]); cmpx(a[5], a[6]);
}
template <class K> __device__ __forceinline__ void bitonic8_desc(K (&a)[8]) {
    cmpx(a[0], a[4]); cmpx(a[1], a[5]); cmpx(a[2], a[6]); cmpx(a[3], a[7]);
    cmpx(a[0], a[2]); cmpx(a[1], a[3]); cmpx(a[4], a[6]); cmpx(a[5], a[7]);
    cmpx(a[0], a[1]); cmpx(a[2], a[3]); cmpx(a[4], a[5]); cmpx(a[6], a[7]);
}
// a, b sorted (descending): a becomes the eight largest of both, sorted
template <class K> __device__ __forceinline__ void merge8_desc(K (&a)[8], const K (&b)[8]) {
#pragma unroll
    for (int i = 0; i < 8; ++i) a[i] = max(a[i], b[7 - i]);
    bitonic8_desc(a);
}

// A key is built in two steps so that its column part costs no arithmetic per element: the column of
// element i of vector v in lane sl is v * LANES * VE + sl * VE + i, three bit fields that do not overlap
// (all powers of two), so the complement 0xffff - col is 0xffff ^ (v * LANES * VE + i) ^ (sl * VE): the
// first part is an immediate folded into the key's last logic operation (local), and the lane's part is
// put into the eight keys that survive the lane's own sort (with_lane). Among one lane's elements the
// local part alone orders equal values by column.
template <int DT> struct RouterKey {                       // 16-bit inputs: value and column in one word
    using type = uint32_t;
    static __device__ __forceinline__ type local(float z, int c) {
        if (DT == DT_BF16) {       // z is a bf16 value (low half of its binary32 image zero): flip the sign bit, or the whole high half
            const uint32_t b = __float_as_uint(z);
            const uint32_t m = (static_cast<uint32_t>(static_cast<int32_t>(b) >> 31) & 0x7fff0000u) | 0x80000000u;
            return b ^ m ^ (0xffffu ^ static_cast<uint32_t>(c));
        }
        const uint32_t h = static_cast<uint32_t>(__half_as_ushort(__float2half_rn(z))); // z is an fp16 value: exact
        const uint32_t o = (h & 0x8000u) ? (~h & 0xffffu) : (h | 0x8000u);
        return (o << 16) | (0xffffu ^ static_cast<uint32_t>(c));
    }
    static __device__ __forceinline__ type with_lane(type k, int lane_cols) { return k ^ static_cast<uint32_t>(lane_cols); }
    static __device__ __forceinline__ int col(type k) { return static_cast<int>(0xffffu - (k & 0xffffu)); }
    static __device__ __forceinline__ float value(type k) {
        const uint32_t o = k >> 16;
        const uint32_t h = (o & 0x8000u) ? (o & 0x7fffu) : (~o & 0xffffu);
        if (DT == DT_BF16) return __uint_as_float(h << 16);
        return __half2float(__ushort_as_half(static_cast<unsigned short>(h)));
    }
};
template <> struct RouterKey<DT_F32> {
    using type = unsigned long long;
    static __device__ __forceinline__ type local(float z, int c) {
        return (static_cast<type>(order_key(z)) << 32) | static_cast<type>(0xffffffffu ^ static_cast<uint32_t>(c));
    }
    static __device__ __forceinline__ type with_lane(type k, int lane_cols) { return k ^ static_cast<type>(static_cast<uint32_t>(lane_cols)); }
    static __device__ __forceinline__ int col(type k) { return static_cast<int>(0xffffffffu - static_cast<uint32_t>(k)); }
    static __device__ __forceinline__ float value(type k) { return order_unkey(static_cast<uint32_t>(k >> 32)); }
};

// FULL: every row has exactly LANES * VPL vectors (no padding keys, no per-vector predicates); the rows
// past the end that the last group of a warp may hold read the last row instead and store nothing.
// The row maximum the softmax needs is not reduced separately: it is the value of the first key once
// the row's eight best are known, so the sum of exponentials follows the selection.
template <int DT, int LANES, int VPL, bool FULL>
__global__ void __launch_bounds__(128)
router_top8_kernel(const RouterParams p) {
    constexpr int VE = Traits<DT>::VE;
    constexpr int G = 32 / LANES;
    constexpr int E = VPL * VE;                            // elements per lane
    constexpr int NG = (E + 7) / 8;                        // groups of eight
    using RK = RouterKey<DT>;
    using K = typename RK::type;
    pdl_launch_dependents();
    const int tid = threadIdx.x, lane = tid & 31;
    const int sub = lane / LANES, sl = lane % LANES;
    const int warps = blockDim.x >> 5;
    const int nvec = static_cast<int>(p.nvec);
    const uint4* __restrict__ xv = static_cast<const uint4*>(p.x);
    const float cabs = fabsf(p.c);
    const float sg = p.c > 0.0f ? 1.0f : (p.c < 0.0f ? -1.0f : 0.0f);
    pdl_wait();

    const int64_t ngroups = (p.rows + G - 1) / G;
    for (int64_t grp = int64_t(blockIdx.x) * warps + (tid >> 5); grp < ngroups; grp += int64_t(gridDim.x) * warps) {
        const int64_t row = grp * G + sub;
        const bool row_ok = row < p.rows;
        const int64_t row_ld = FULL ? (row_ok ? row : p.rows - 1) : row;
        float z[VPL][VE];
        bool live[VPL];
#pragma unroll
        for (int v = 0; v < VPL; ++v) {
            live[v] = FULL || (row_ok && sl + v * LANES < nvec);
            uint4 raw = make_uint4(0u, 0u, 0u, 0u);
            if (live[v]) raw = ld_stream(xv + row_ld * p.nvec + sl + v * LANES);
            unpack<DT>(raw, z[v]);
#pragma unroll
            for (int i = 0; i < VE; ++i) z[v][i] = fmaf(z[v][i], sg, 0.0f);   // sign of the scale; -0 becomes +0; inf * 0 = NaN
        }

        // ---- this lane's eight best
        K best[8];
#pragma unroll
        for (int g = 0; g < NG; ++g) {
            K grp8[8];
#pragma unroll
            for (int j = 0; j < 8; ++j) {
                const int f = g * 8 + j;                   // flat element of this lane
                grp8[j] = 0;
                if (f < E) {
                    const int v = f / VE, i = f % VE;
                    const float kz = fmaxf(z[v][i], __int_as_float(0xff800000));       // NaN counts as -inf (fmaxf drops it)
                    const K key = RK::local(kz, v * LANES * VE + i);
                    grp8[j] = (FULL || live[v]) ? key : K(0);                            // padding is never selected
                }
            }
            sort8_desc(grp8);
            if (g == 0) {
#pragma unroll
                for (int j = 0; j < 8; ++j) best[j] = grp8[j];
            } else {
                merge8_desc(best, grp8);
            }
        }
#pragma unroll
        for (int j = 0; j < 8; ++j) best[j] = RK::with_lane(best[j], sl * VE);
        // ---- the row's eight best: merge across the lanes of the group
#pragma unroll
        for (int o = 1; o < LANES; o <<= 1) {
            K other[8];
#pragma unroll
            for (int j = 0; j < 8; ++j) other[j] = __shfl_xor_sync(0xffffffffu, best[j], o);
            merge8_desc(best, other);
        }
        // ---- the softmax sum against the row maximum (the first key; -inf for a row of NaN or -inf only)
        const float key0 = RK::value(best[0]);
        float s = 0.0f;
#pragma unroll
        for (int v = 0; v < VPL; ++v)
#pragma unroll
            for (int i = 0; i < VE; ++i)
                if (FULL || live[v]) s += ex2_ftz_r((z[v][i] - key0) * cabs);
        s = warp_sum<LANES>(s);
        const float inv_s = 1.0f / s;                      // NaN when the row is NaN
        // ---- weights and output: entry r by lane r mod LANES
        float e[8];
        float sel = 0.0f;
#pragma unroll
        for (int r = 0; r < 8; ++r) {
            e[r] = ex2_ftz_r((RK::value(best[r]) - key0) * cabs);
            if (r < p.k) sel += e[r];
        }
        // 0 * inv_s carries a NaN row into the renormalised weights (inv_s is finite otherwise)
        const float f = p.renorm ? 1.0f / sel + 0.0f * inv_s : inv_s;
        if (p.wide) {
            // every lane of the group holds the whole list: one lane stores the row's 32 bytes of weights, another
            // its 32 bytes of columns (whole sectors, two store instructions instead of sixteen partial ones)
            if (row_ok && sl == 0)
                st_stream32(reinterpret_cast<uint4*>(p.w + row * 8),
                            make_uint4(__float_as_uint(e[0] * f), __float_as_uint(e[1] * f), __float_as_uint(e[2] * f), __float_as_uint(e[3] * f)),
                            make_uint4(__float_as_uint(e[4] * f), __float_as_uint(e[5] * f), __float_as_uint(e[6] * f), __float_as_uint(e[7] * f)));
            if (row_ok && sl == (LANES > 1 ? 1 : 0))
                st_stream32(reinterpret_cast<uint4*>(p.idx + row * 8),
                            make_uint4(uint32_t(RK::col(best[0])), uint32_t(RK::col(best[1])), uint32_t(RK::col(best[2])), uint32_t(RK::col(best[3]))),
                            make_uint4(uint32_t(RK::col(best[4])), uint32_t(RK::col(best[5])), uint32_t(RK::col(best[6])), uint32_t(RK::col(best[7]))));
        } else {
#pragma unroll
            for (int r = 0; r < 8; ++r) {
                if (row_ok && r < p.k && (r % LANES) == sl) {
                    p.idx[row * p.k + r] = RK::col(best[r]);
                    p.w[row * p.k + r] = e[r] * f;
                }
            }
        }
    }
}

}  // namespace fsm
