// Kernels that form their output from x itself, so nothing is written back over the resident row:
//   OUT_LOG    log_softmax: y = z - max z - ln sum exp(z - max z), z = scale * x, in x's dtype
//                  d = x - r,  S = sum 2^(d c),  y = d * scale - ln S      (c = scale * log2 e)
//   OUT_PROB32 softmax of a 16-bit tensor written as binary32 (what eager attention asks for with
//              softmax(..., dtype=float32)): y = 2^(d c) / S, the exponential taken a second time
// The same skeleton as the softmax kernels (one read, reduce, one write).
// A negative scale is folded into the data: the sign bit of every element is flipped on load and
// |scale| is used, which is the same product exactly; the kernels therefore always look for a
// maximum.
//
//   lsm_warp_kernel     (sub-)warp per row, the row packed in registers (rows up to 9 KiB)
//   lsm_tile_kernel     rows of 4-12 KiB: four rows per block in shared memory, a warp per row
//   lsm_smem_kernel     row split over a cluster of 1..16 blocks, slices resident in shared memory
//                       (bulk async copies, per-chunk mbarriers, online (max, sum) per thread,
//                       pairs merged warp -> block -> cluster through st.async); pass 2 reads the
//                       untouched slice again
//   lsm_generic_kernel  block per row, element-wise, any shape and alignment
#pragma once
#include "block_row.cuh"
#include "common.cuh"
#include "norm_row.cuh"

namespace fsm {

enum : int { OUT_LOG = 0, OUT_PROB32 = 1 };

struct LsmParams {
    const void* x;
    void* y;
    int64_t rows;
    int64_t cols;
    int64_t nvec;
    float c;            // |scale| * log2(e)
    float scale;        // |scale|
    uint32_t flip;      // XOR mask per 32-bit word that negates every element (0 for scale >= 0)
    int* status;
    int64_t pf_rows;
    float lag_ns;          // first wave of a one-shot grid: cluster i < lag_rows starts i * lag_ns late
    int lag_rows;
    int early_pf;          // first wave: ask L2 for the block's own input before griddepcontrol.wait (pdl_early_prefetch)
    int wide;              // OUT_PROB32: y is 32-byte aligned, a vector's eight floats leave in one 256-bit store
};

__device__ __forceinline__ float lg2_approx(float v) {
    float r;
    asm("lg2.approx.f32 %0, %1;" : "=f"(r) : "f"(v));
    return r;
}
// ln S from the special-function unit's log2 (absolute error about 2^-22 for S >= 1)
__device__ __forceinline__ float ln_of(float s) { return lg2_approx(s) * 0.6931471805599453f; }

__device__ __forceinline__ uint4 flip_vec(uint4 v, uint32_t m) {
    v.x ^= m; v.y ^= m; v.z ^= m; v.w ^= m;
    return v;
}

// d = x - r for one vector, S += 2^(d c) pairwise; d is kept as pairs.
template <int DT>
__device__ __forceinline__ void lsm_accumulate(const uint4& raw, f32x2 r2, f32x2 c2, f32x2 (&d)[Traits<DT>::VE / 2], f32x2 (&acc)[2]) {
    constexpr int NP = Traits<DT>::VE / 2;
    widen_pairs<DT>(raw, d);
#pragma unroll
    for (int k = 0; k < NP; ++k) {
        d[k] = sub2(d[k], r2);
        float lo, hi;
        unpair(mul2(d[k], c2), lo, hi);
        acc[k & 1] = add2(acc[k & 1], pair(ex2_ftz(lo), ex2_ftz(hi)));
    }
}

// One vector of output from one (sign-adjusted) vector of x. `ybase` is the row's first output
// element; `v` the vector's index in the row. k2 is -ln S (OUT_LOG) or 1/S (OUT_PROB32).
// wide (OUT_PROB32, y 32-byte aligned): the vector's eight floats leave in one 256-bit store.
template <int DT, int OUT>
__device__ __forceinline__ void lsm_emit(const uint4& raw, f32x2 r2, f32x2 c2, f32x2 s2, f32x2 k2, void* ybase, int64_t v, bool wide) {
    constexpr int NP = Traits<DT>::VE / 2;
    f32x2 d[NP];
    widen_pairs<DT>(raw, d);
    if constexpr (OUT == OUT_LOG) {
#pragma unroll
        for (int j = 0; j < NP; ++j) d[j] = fma2(sub2(d[j], r2), s2, k2);
        st_stream(static_cast<uint4*>(ybase) + v, narrow_pairs<DT>(d));
    } else {
        static_assert(OUT == OUT_LOG || DT != DT_F32, "binary32 output is for 16-bit inputs");
#pragma unroll
        for (int j = 0; j < NP; ++j) {
            float lo, hi;
            unpair(mul2(sub2(d[j], r2), c2), lo, hi);
            d[j] = mul2(pair(ex2_ftz(lo), ex2_ftz(hi)), k2);
        }
        uint4* out = static_cast<uint4*>(ybase) + 2 * v;              // eight floats: two vectors
        uint4 a, b;
        unpair_bits(d[0], a.x, a.y); unpair_bits(d[1], a.z, a.w);
        unpair_bits(d[NP - 2], b.x, b.y); unpair_bits(d[NP - 1], b.z, b.w);
        if (wide) {
            st_stream32(out, a, b);
        } else {
            st_stream(out, a);
            st_stream(out + 1, b);
        }
    }
}

// ---------------------------------------------------------------------------------------------
template <int DT, int LANES, int VPL, int OUT>
__device__ __forceinline__ void lsm_warp_body(const LsmParams& p) {
    constexpr int NP = Traits<DT>::VE / 2;
    constexpr int G = 32 / LANES;
    pdl_launch_dependents();
    const int lane = threadIdx.x & 31;
    const int sub = lane / LANES, sl = lane % LANES;
    const int warps = blockDim.x >> 5;
    const int nvec = static_cast<int>(p.nvec);
    const uint4* __restrict__ xv = static_cast<const uint4*>(p.x);
    const int64_t ypitch = OUT == OUT_LOG ? p.nvec * 16 : p.cols * 4;      // bytes per output row
    const f32x2 c2 = pair(p.c, p.c), s2 = pair(p.scale, p.scale);
    pdl_wait();
    const int64_t ngroups = (p.rows + G - 1) / G;
    for (int64_t grp = int64_t(blockIdx.x) * warps + (threadIdx.x >> 5); grp < ngroups; grp += int64_t(gridDim.x) * warps) {
        const int64_t row = grp * G + sub;
        const bool row_ok = row < p.rows;
        uint4 raw[VPL];
        RefAcc<DT, false> ref;
        ref.init();
#pragma unroll
        for (int k = 0; k < VPL; ++k) {
            raw[k] = make_uint4(0u, 0u, 0u, 0u);
            if (row_ok && sl + k * LANES < nvec) {
                raw[k] = flip_vec(ld_stream(xv + row * p.nvec + sl + k * LANES), p.flip);
                ref.fold(raw[k]);
            }
        }
        const float r = warp_pick<LANES, false>(ref.value());
        const f32x2 r2 = pair(r, r);
        // the row stays packed in registers and is widened where it is used (twice): a widened row
        // of eight vectors per lane costs 64 more registers and a third of the resident warps
        f32x2 acc[2] = {pair(0.0f, 0.0f), pair(0.0f, 0.0f)};
#pragma unroll
        for (int k = 0; k < VPL; ++k) {
            if (sl + k * LANES < nvec) {
                f32x2 d[NP];
                lsm_accumulate<DT>(raw[k], r2, c2, d, acc);
            }
        }
        const float ssum = warp_sum<LANES>(pair_sum(add2(acc[0], acc[1])));
        const float kk = OUT == OUT_LOG ? -ln_of(ssum) : 1.0f / ssum;
        const f32x2 k2 = pair(kk, kk);
        if (row_ok) {
            char* yrow = static_cast<char*>(p.y) + row * ypitch;
#pragma unroll
            for (int k = 0; k < VPL; ++k)
                if (sl + k * LANES < nvec) lsm_emit<DT, OUT>(raw[k], r2, c2, s2, k2, yrow, sl + k * LANES, p.wide != 0);
        }
    }
}

// Up to eight vectors per lane the compiler's own register choice is best (an explicit minimum of
// blocks per SM, even 1, makes it spend registers: measured 88 us against 80 on short rows); the
// long-row variants are capped so that four or five blocks stay resident.
template <int DT, int LANES, int VPL, int OUT>
__global__ void __launch_bounds__(128)
lsm_warp_kernel(const LsmParams p) {
    lsm_warp_body<DT, LANES, VPL, OUT>(p);
}
template <int DT, int VPL, int OUT>
__global__ void __launch_bounds__(128, VPL <= 12 ? 5 : 4)
lsm_warp_long_kernel(const LsmParams p) {
    lsm_warp_body<DT, 32, VPL, OUT>(p);
}

// ---------------------------------------------------------------------------------------------
// Rows of 4-11 KiB: four rows per block, each brought to shared memory by a bulk copy of its own
// (one mbarrier per row) and worked on by one warp alone with the arithmetic of the warp kernel
// above (three reads of shared memory: reference, sum, output); no block barrier after start-up.
// One-shot grid: block b handles rows b*W .. b*W+W-1. dynamic shared memory: W rows | W mbarriers
// ---------------------------------------------------------------------------------------------
template <int DT, int OUT>
__global__ void __launch_bounds__(128)
lsm_tile_kernel(const LsmParams p) {
    constexpr int NP = Traits<DT>::VE / 2;
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
    const uint4* sv = reinterpret_cast<const uint4*>(smem + size_t(w) * size_t(row_bytes)) + lane;
    const int64_t ypitch = OUT == OUT_LOG ? p.nvec * 16 : p.cols * 4;      // bytes per output row
    char* yrow = static_cast<char*>(p.y) + row * ypitch;
    const f32x2 c2 = pair(p.c, p.c), s2 = pair(p.scale, p.scale);
    mbar_wait_warp(smem_u32(&bars[w]), 0u, p.status);      // on a timeout the status word is set and the row is garbage

    RefAcc<DT, false> ref;
    ref.init();
    for (int k0 = 0; k0 < nvec; k0 += 32 * H) {
#pragma unroll
        for (int u = 0; u < H; ++u)
            if (k0 + u * 32 + lane < nvec) ref.fold(flip_vec(sv[k0 + u * 32], p.flip));
    }
    const float r = warp_pick<32, false>(ref.value());
    const f32x2 r2 = pair(r, r);
    f32x2 acc[2] = {pair(0.0f, 0.0f), pair(0.0f, 0.0f)};
    for (int k0 = 0; k0 < nvec; k0 += 32 * H) {
        uint4 raw[H];
#pragma unroll
        for (int u = 0; u < H; ++u) {
            raw[u] = make_uint4(0u, 0u, 0u, 0u);
            if (k0 + u * 32 + lane < nvec) raw[u] = flip_vec(sv[k0 + u * 32], p.flip);
        }
#pragma unroll
        for (int u = 0; u < H; ++u) {
            if (k0 + u * 32 + lane < nvec) {
                f32x2 d[NP];
                lsm_accumulate<DT>(raw[u], r2, c2, d, acc);
            }
        }
    }
    const float ssum = warp_sum<32>(pair_sum(add2(acc[0], acc[1])));
    const float kk = OUT == OUT_LOG ? -ln_of(ssum) : 1.0f / ssum;
    const f32x2 k2 = pair(kk, kk);
    for (int k0 = 0; k0 < nvec; k0 += 32 * H) {
        uint4 raw[H];
#pragma unroll
        for (int u = 0; u < H; ++u) {
            raw[u] = make_uint4(0u, 0u, 0u, 0u);
            if (k0 + u * 32 + lane < nvec) raw[u] = flip_vec(sv[k0 + u * 32], p.flip);
        }
#pragma unroll
        for (int u = 0; u < H; ++u)
            if (k0 + u * 32 + lane < nvec) lsm_emit<DT, OUT>(raw[u], r2, c2, s2, k2, yrow, k0 + u * 32 + lane, p.wide != 0);
    }
}

// ---------------------------------------------------------------------------------------------
// cluster per row (one-shot grid: cluster i handles row i); dynamic shared memory: slice rounded
// up to whole chunks (stage_bytes) | 8 chunk mbarriers
// ---------------------------------------------------------------------------------------------
template <int DT, bool FULL, int OUT>
__global__ void __launch_bounds__(256, 3)
lsm_smem_kernel(const LsmParams p, const uint32_t stage_bytes, const int slice, const int nchunk_full) {
    constexpr int VE = Traits<DT>::VE;
    constexpr int NP = VE / 2;
    constexpr int U = 8;
    pdl_launch_dependents();
    extern __shared__ __align__(128) unsigned char smem[];
    __shared__ float2 wp[2][32];
    __shared__ __align__(16) float2 xchg[16];
    __shared__ __align__(8) uint64_t xbar;
    const int T = blockDim.x, tid = threadIdx.x, lane = tid & 31;
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
    const float ident = ref_identity<false>();
    uint64_t* bars = reinterpret_cast<uint64_t*>(smem + stage_bytes);
    const uint4* sv = reinterpret_cast<const uint4*>(smem) + tpos;
    const int64_t row_bytes = p.nvec * 16;
    const char* xb = static_cast<const char*>(p.x) + int64_t(v0) * 16;
    const f32x2 c2 = pair(p.c, p.c);

    if (tid == 0) {
        for (int ch = 0; ch < kNormMaxChunks; ++ch) mbar_init(smem_u32(&bars[ch]), 1);
        mbar_init(smem_u32(&xbar), 1);
        mbar_fence_init();
        fence_proxy_async_smem();
        pdl_wait_first_wave<true>(row, p.lag_ns, p.lag_rows, p.early_pf, [&] { if (nv > 0) { pdl_early_prefetch(xb + row * row_bytes, int64_t(nv) * 16); } });
        for (int ch = 0; ch < nchunk; ++ch) {
            const int cv = FULL ? chunk_vecs : min(chunk_vecs, nv - ch * chunk_vecs);
            bulk_load_row(smem_u32(smem) + uint32_t(ch) * uint32_t(chunk_vecs) * 16u,
                          xb + row * row_bytes + int64_t(ch) * chunk_vecs * 16, uint32_t(cv) * 16u, smem_u32(&bars[ch]));
        }
        if (p.pf_rows > 0 && row + p.pf_rows < p.rows && nv > 0)
            l2_prefetch(xb + (row + p.pf_rows) * row_bytes, uint32_t(nv) * 16u);
        if (cs > 1) mbar_expect_tx(smem_u32(&xbar), cs * 8u);
    }
    __syncthreads();
    if (cs > 1) {
        cluster_arrive_relaxed();
        cluster_wait_acquire();
    }
    pdl_wait();

    // ---- pass 1: online (reference, sum) over the chunks as they land
    bool alive = true;
    float r = ident, s = 0.0f;
    const uint32_t idw = ident_word<DT, false>() ^ p.flip;       // flips back to the identity when loaded
    for (int ch = 0; ch < nchunk; ++ch) {
        if (tid < 32 && alive) alive = mbar_wait_warp(smem_u32(&bars[ch]), 0u, p.status);
        if (T > 32) __syncthreads();
        const uint4* sc = sv + ch * chunk_vecs;
        const int cbase = ch * chunk_vecs + tpos;
        uint4 raw[U];
        RefAcc<DT, false> ref;
        ref.init();
#pragma unroll
        for (int u = 0; u < U; ++u) {
            raw[u] = sc[u * 32];
            if (!FULL && cbase + u * 32 >= nv) raw[u] = make_uint4(idw, idw, idw, idw);    // past the slice: drops out
            raw[u] = flip_vec(raw[u], p.flip);
            ref.fold(raw[u]);
        }
        const float rc = ref.value();
        const float ru = (rc == ident) ? 0.0f : rc;
        const f32x2 ru2 = pair(ru, ru);
        f32x2 acc[2] = {pair(0.0f, 0.0f), pair(0.0f, 0.0f)};
#pragma unroll
        for (int u = 0; u < U; ++u) {
            f32x2 d[NP];
            lsm_accumulate<DT>(raw[u], ru2, c2, d, acc);
        }
        const float part = pair_sum(add2(acc[0], acc[1]));
        const float rn = fmaxf(r, rc);
        const bool keep = (rn == r);
        const float lo = keep ? rc : r;
        const float f = (lo == ident) ? 1.0f : ex2_ftz((lo - rn) * p.c);
        s = keep ? fmaf(part, f, s) : fmaf(s, f, part);
        r = rn;
    }
    float R = r;
    block_merge_pairs<false>(R, s, wp[0], p.c);
    if (cs > 1) {
        if (tid < cs) st_async_v2(map_to_rank(smem_u32(&xchg[q]), tid), R, s, map_to_rank(smem_u32(&xbar), tid));
        cluster_arrive_relaxed();          // exit guard: waited for after pass 2 (see smem_row.cuh)
        if (tid < 32 && alive) alive = mbar_wait_warp(smem_u32(&xbar), 0u, p.status);
        if (T > 32) __syncthreads();
        R = ident; s = 0.0f;
        if (lane < static_cast<int>(cs)) ld_shared_v2(smem_u32(&xchg[lane]), R, s);
        warp_merge_pairs<false>(R, s, p.c);
    }
    const float kk = OUT == OUT_LOG ? -ln_of(s) : 1.0f / s;

    // ---- pass 2: the output from the resident, untouched slice
    const f32x2 R2 = pair(R, R), s2 = pair(p.scale, p.scale), k2 = pair(kk, kk);
    char* yrow = static_cast<char*>(p.y) + row * (OUT == OUT_LOG ? p.nvec * 16 : p.cols * 4);
    for (int ch = 0; ch < nchunk; ++ch) {
        const uint4* sc = sv + ch * chunk_vecs;
        const int cbase = ch * chunk_vecs + tpos;
        uint4 raw[U];
#pragma unroll
        for (int u = 0; u < U; ++u) raw[u] = sc[u * 32];
#pragma unroll
        for (int u = 0; u < U; ++u) {
            if (FULL || cbase + u * 32 < nv)
                lsm_emit<DT, OUT>(flip_vec(raw[u], p.flip), R2, c2, s2, k2, yrow, int64_t(v0) + cbase + u * 32, p.wide != 0);
        }
    }
    if (cs > 1) cluster_wait_acquire();    // no block leaves while a peer's deposit into it is still to be issued
}

// ---------------------------------------------------------------------------------------------
template <int DT, int OUT>
__global__ void __launch_bounds__(1024)
lsm_generic_kernel(const LsmParams p) {
    __shared__ float red[32];
    pdl_launch_dependents();
    pdl_wait();
    const float sg = p.flip ? -1.0f : 1.0f;
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5, nwarps = blockDim.x >> 5;
    for (int64_t row = blockIdx.x; row < p.rows; row += gridDim.x) {
        const int64_t base = row * p.cols;
        float m = ref_identity<false>();
        for (int64_t j = threadIdx.x; j < p.cols; j += blockDim.x) m = fmaxf(m, load_elem<DT>(p.x, base + j) * sg);
        m = warp_pick<32, false>(m);
        __syncthreads();
        if (lane == 0) red[warp] = m;
        __syncthreads();
        m = warp_pick<32, false>(lane < nwarps ? red[lane] : ref_identity<false>());
        float s = 0.0f;
        for (int64_t j = threadIdx.x; j < p.cols; j += blockDim.x)
            s += ex2_ftz((load_elem<DT>(p.x, base + j) * sg - m) * p.c);
        const float ssum = block_sum(s, red);
        if (OUT == OUT_LOG) {
            const float lns = ln_of(ssum);
            for (int64_t j = threadIdx.x; j < p.cols; j += blockDim.x)
                store_elem<DT>(p.y, base + j, fmaf(load_elem<DT>(p.x, base + j) * sg - m, p.scale, -lns));
        } else {
            const float inv = 1.0f / ssum;
            for (int64_t j = threadIdx.x; j < p.cols; j += blockDim.x)
                static_cast<float*>(p.y)[base + j] = ex2_ftz((load_elem<DT>(p.x, base + j) * sg - m) * p.c) * inv;
        }
    }
}

}  // namespace fsm
