// Row normalisations: layer_norm over the last dimension and group_norm over (sample, group)
// blocks of an [n, channels, spatial] tensor, which is the same computation on rows of
// channels/groups * spatial elements with the affine parameters indexed by channel:
//     mu = mean x,  var = mean (x - mu)^2 (biased),  y = (x - mu) / sqrt(var + eps) * gamma + beta
// The skeleton is the softmax kernels' (load once, reduce, rescale, store once); the reduction
// item is the triple (n, mean, M2) with Chan's pairwise merge in place of the (reference, sum) pair.
//
//   norm_warp_kernel     (sub-)warp per row, the row in registers: exact two-pass statistics
//   norm_tile_kernel     rows of 4-11 KiB: four rows per block, each brought to shared memory by a
//                        bulk copy of its own and worked on by one warp (three reads of shared memory)
//   norm_smem_kernel     row split over a cluster of 1..16 blocks, the slice resident in shared
//                        memory (bulk async copies, one mbarrier per chunk); per chunk a thread
//                        takes the exact mean and M2 of its own 8 vectors and merges them into
//                        its running triple; triples merge warp -> block -> cluster (st.async
//                        deposits counted by an mbarrier); pass 2 normalises from shared memory
//   norm_partial_kernel + norm_apply_kernel   few, very long rows: segments of a row on separate
//                        blocks, partial triples exchanged through global memory between the two
//   norm_generic_kernel  block per row, three passes over global memory (the later ones normally
//                        from L2): any column count, alignment and row length
//
// AFF: 0 no affine parameters, 1 one (gamma, beta) per column (layer_norm: vectors loaded like x),
//      2 one per run of `run_vecs` vectors (group_norm: a channel's spatial extent).
#pragma once
#include "common.cuh"

namespace fsm {

struct NormParams {
    const void* x;
    void* y;
    const void* gamma;     // may be null (1)
    const void* beta;      // may be null (0)
    int64_t rows;
    int64_t cols;
    int64_t nvec;          // 16-byte vectors per row (fast kernels)
    float eps;
    int64_t run_elems;     // AFF 2: elements per affine entry (spatial); 1 otherwise
    int64_t aff_rows;      // AFF 2: rows per sample (groups): row % aff_rows selects the channel block
    int* status;
    int64_t pf_rows;       // one-shot grids: L2 prefetch distance in rows (0: off)
    float lag_ns;          // first wave of a one-shot grid: cluster i < lag_rows starts i * lag_ns late
    int lag_rows;
    int early_pf;          // first wave: ask L2 for the block's own input before griddepcontrol.wait (pdl_early_prefetch)
};

// (count, mean, sum of squared deviations)
struct Stat { float n, mean, m2; };

// Chan's pairwise merge. The weight b.n / n only positions the merged mean between the two
// means, so the special-function unit's reciprocal (1 ulp) is enough; an IEEE division would cost
// more instructions than the rest of the merge.
__device__ __forceinline__ float fast_rcp(float v) {
    float r;
    asm("rcp.approx.ftz.f32 %0, %1;" : "=f"(r) : "f"(v));
    return r;
}
__device__ __forceinline__ Stat stat_merge(const Stat& a, const Stat& b) {
    Stat r;
    r.n = a.n + b.n;
    const float w = r.n > 0.0f ? b.n * fast_rcp(r.n) : 0.0f;
    const float d = b.mean - a.mean;
    r.mean = fmaf(d, w, a.mean);
    r.m2 = a.m2 + b.m2 + d * d * a.n * w;
    return r;
}

template <int WIDTH>
__device__ __forceinline__ Stat warp_merge_stats(Stat s) {
#pragma unroll
    for (int o = WIDTH / 2; o > 0; o >>= 1) {
        Stat t;
        t.n = __shfl_xor_sync(0xffffffffu, s.n, o);
        t.mean = __shfl_xor_sync(0xffffffffu, s.mean, o);
        t.m2 = __shfl_xor_sync(0xffffffffu, s.m2, o);
        s = stat_merge(s, t);
    }
    return s;
}

// 1 / sqrt(var + eps): the special-function unit's reciprocal square root (relative error 2^-22)
// and one Newton step, which brings it to about one unit in the last place.
__device__ __forceinline__ float rstd_of(float var, float eps) {
    const float v = var + eps;
    float r;
    asm("rsqrt.approx.f32 %0, %1;" : "=f"(r) : "f"(v));
    const float h = 0.5f * v * r;
    const float refined = fmaf(r, fmaf(-h, r, 0.5f), r);      // r + r (1/2 - v r^2 / 2)
    return (v > 0.0f && v < __int_as_float(0x7f800000)) ? refined : r;   // 0, inf, NaN: keep the unit's answer
}

__device__ __forceinline__ uint4 ld_cached(const uint4* p) {
    FS_DBG_LOAD(p, 16, make_uint4(0u, 0u, 0u, 0u));
    uint4 v;
    asm volatile("ld.global.nc.v4.u32 {%0,%1,%2,%3}, [%4];" : "=r"(v.x), "=r"(v.y), "=r"(v.z), "=r"(v.w) : "l"(p));
    return v;
}

// One vector of x as pairs of binary32.
template <int DT>
__device__ __forceinline__ void widen_pairs(const uint4& raw, f32x2 (&x)[Traits<DT>::VE / 2]) {
    if constexpr (DT == DT_F32) {
        x[0] = pair_bits(raw.x, raw.y); x[1] = pair_bits(raw.z, raw.w);
    } else {
        x[0] = widen_word<DT>(raw.x); x[1] = widen_word<DT>(raw.y);
        x[2] = widen_word<DT>(raw.z); x[3] = widen_word<DT>(raw.w);
    }
}
template <int DT>
__device__ __forceinline__ uint4 narrow_pairs(const f32x2 (&x)[Traits<DT>::VE / 2]) {
    uint4 v;
    if constexpr (DT == DT_F32) {
        unpair_bits(x[0], v.x, v.y); unpair_bits(x[1], v.z, v.w);
    } else {
        uint32_t o[4];
#pragma unroll
        for (int k = 0; k < 4; ++k) {
            float lo, hi;
            unpair(x[k], lo, hi);
            o[k] = DT == DT_BF16 ? pack_bf16x2(lo, hi) : pack_f16x2(lo, hi);
        }
        v = make_uint4(o[0], o[1], o[2], o[3]);
    }
    return v;
}

// Centred pairs d = x - mu of one vector -> d * rstd [* gamma] [+ beta], rounded and stored.
// Which parameters exist is a compile-time choice here: a run-time "if (gamma)" per element turns
// into two select instructions per pair, which cost more than the arithmetic.
template <int DT, bool HG, bool HB>
__device__ __forceinline__ void affine_store(f32x2 (&d)[Traits<DT>::VE / 2], f32x2 r2, const uint4& graw, const uint4& braw, uint4* dst) {
    constexpr int NP = Traits<DT>::VE / 2;
    f32x2 g[NP], b[NP];
    if (HG) widen_pairs<DT>(graw, g);
    if (HB) widen_pairs<DT>(braw, b);
#pragma unroll
    for (int j = 0; j < NP; ++j) {
        f32x2 t = mul2(d[j], r2);
        if (HG && HB) t = fma2(t, g[j], b[j]);
        else if (HG) t = mul2(t, g[j]);
        else if (HB) t = add2(t, b[j]);
        d[j] = t;
    }
    st_stream(dst, narrow_pairs<DT>(d));
}
template <int DT>
__device__ __forceinline__ void affine_store_any(bool hg, bool hb, f32x2 (&d)[Traits<DT>::VE / 2], f32x2 r2, const uint4& graw,
                                                 const uint4& braw, uint4* dst) {
    if (hg && hb) affine_store<DT, true, true>(d, r2, graw, braw, dst);
    else if (hg)  affine_store<DT, true, false>(d, r2, graw, braw, dst);
    else if (hb)  affine_store<DT, false, true>(d, r2, graw, braw, dst);
    else          affine_store<DT, false, false>(d, r2, graw, braw, dst);
}

// ---------------------------------------------------------------------------------------------
// (sub-)warp per row, registers
// ---------------------------------------------------------------------------------------------
template <int DT, int LANES, int VPL, int AFF>
__global__ void __launch_bounds__(128)
norm_warp_kernel(const NormParams p) {
    constexpr int NP = Traits<DT>::VE / 2;
    constexpr int G = 32 / LANES;
    static_assert(AFF != 2, "per-run affine parameters are handled by the shared-memory kernel");
    pdl_launch_dependents();
    const int lane = threadIdx.x & 31;
    const int sub = lane / LANES, sl = lane % LANES;
    const int warps = blockDim.x >> 5;
    const int nvec = static_cast<int>(p.nvec);
    const uint4* __restrict__ xv = static_cast<const uint4*>(p.x);
    uint4* __restrict__ yv = static_cast<uint4*>(p.y);
    const uint4* gv = AFF == 1 && p.gamma ? static_cast<const uint4*>(p.gamma) + sl : nullptr;
    const uint4* bv = AFF == 1 && p.beta ? static_cast<const uint4*>(p.beta) + sl : nullptr;
    const float inv_n = 1.0f / static_cast<float>(p.cols);
    pdl_wait();
    const int64_t ngroups = (p.rows + G - 1) / G;
    for (int64_t grp = int64_t(blockIdx.x) * warps + (threadIdx.x >> 5); grp < ngroups; grp += int64_t(gridDim.x) * warps) {
        const int64_t row = grp * G + sub;
        const bool row_ok = row < p.rows;
        const uint4* xr = xv + row * p.nvec + sl;
        uint4 raw[VPL];
#pragma unroll
        for (int k = 0; k < VPL; ++k) {
            raw[k] = make_uint4(0u, 0u, 0u, 0u);
            if (row_ok && sl + k * LANES < nvec) raw[k] = ld_stream(xr + k * LANES);
        }
        f32x2 x[VPL][NP];
        f32x2 acc[2] = {pair(0.0f, 0.0f), pair(0.0f, 0.0f)};
#pragma unroll
        for (int k = 0; k < VPL; ++k) {
            widen_pairs<DT>(raw[k], x[k]);                                  // absent vectors are zeros
#pragma unroll
            for (int j = 0; j < NP; ++j) acc[j & 1] = add2(acc[j & 1], x[k][j]);
        }
        const float mu = warp_sum<LANES>(pair_sum(add2(acc[0], acc[1]))) * inv_n;
        const f32x2 mu2 = pair(mu, mu);
        acc[0] = pair(0.0f, 0.0f); acc[1] = pair(0.0f, 0.0f);
#pragma unroll
        for (int k = 0; k < VPL; ++k) {
            if (sl + k * LANES < nvec) {
#pragma unroll
                for (int j = 0; j < NP; ++j) { x[k][j] = sub2(x[k][j], mu2); acc[j & 1] = fma2(x[k][j], x[k][j], acc[j & 1]); }
            }
        }
        const float rstd = rstd_of(warp_sum<LANES>(pair_sum(add2(acc[0], acc[1]))) * inv_n, p.eps);
        const f32x2 r2 = pair(rstd, rstd);
        if (row_ok) {
            uint4* yr = yv + row * p.nvec + sl;
#pragma unroll
            for (int k = 0; k < VPL; ++k) {
                if (sl + k * LANES < nvec) {
                    uint4 graw = make_uint4(0u, 0u, 0u, 0u), braw = make_uint4(0u, 0u, 0u, 0u);
                    if (gv) graw = ld_cached(gv + k * LANES);
                    if (bv) braw = ld_cached(bv + k * LANES);
                    affine_store_any<DT>(gv != nullptr, bv != nullptr, x[k], r2, graw, braw, yr + k * LANES);
                }
            }
        }
    }
}

// ---------------------------------------------------------------------------------------------
// warp per row FROM SHARED MEMORY (rows of 4-16 KiB): a block of W warps brings W consecutive rows
// with one bulk copy each, every copy on an mbarrier of its own, and each warp works on its row
// alone: three reads of shared memory (sum, squared deviations, output), no block barrier after
// start-up, and a register footprint that does not grow with the row, so that many warps are
// resident. One-shot grid: block b handles rows b*W .. b*W+W-1.
// dynamic shared memory: W rows | W mbarriers
// ---------------------------------------------------------------------------------------------
template <int DT, int AFF>
__global__ void __launch_bounds__(128)
norm_tile_kernel(const NormParams p) {
    constexpr int NP = Traits<DT>::VE / 2;
    constexpr int H = 4;                                   // vectors per lane and batch
    static_assert(AFF != 2, "per-run affine parameters are handled by the split-row kernel");
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
    uint4* __restrict__ yv = static_cast<uint4*>(p.y) + row * p.nvec + lane;
    const uint4* gv = AFF == 1 && p.gamma ? static_cast<const uint4*>(p.gamma) + lane : nullptr;
    const uint4* bv = AFF == 1 && p.beta ? static_cast<const uint4*>(p.beta) + lane : nullptr;
    const float inv_n = 1.0f / static_cast<float>(p.cols);
    mbar_wait_warp(smem_u32(&bars[w]), 0u, p.status);      // on a timeout the status word is set and the row is garbage

    f32x2 acc[2] = {pair(0.0f, 0.0f), pair(0.0f, 0.0f)};
    for (int k0 = 0; k0 < nvec; k0 += 32 * H) {
        uint4 raw[H];
#pragma unroll
        for (int u = 0; u < H; ++u) {
            raw[u] = make_uint4(0u, 0u, 0u, 0u);           // absent vectors are zeros: they add nothing
            if (k0 + u * 32 + lane < nvec) raw[u] = sv[k0 + u * 32];
        }
#pragma unroll
        for (int u = 0; u < H; ++u) {
            f32x2 x[NP];
            widen_pairs<DT>(raw[u], x);
#pragma unroll
            for (int j = 0; j < NP; ++j) acc[j & 1] = add2(acc[j & 1], x[j]);
        }
    }
    const float mu = warp_sum<32>(pair_sum(add2(acc[0], acc[1]))) * inv_n;
    const f32x2 mu2 = pair(mu, mu);
    acc[0] = pair(0.0f, 0.0f); acc[1] = pair(0.0f, 0.0f);
    for (int k0 = 0; k0 < nvec; k0 += 32 * H) {
        uint4 raw[H];
#pragma unroll
        for (int u = 0; u < H; ++u) {
            raw[u] = make_uint4(0u, 0u, 0u, 0u);
            if (k0 + u * 32 + lane < nvec) raw[u] = sv[k0 + u * 32];
        }
#pragma unroll
        for (int u = 0; u < H; ++u) {
            if (k0 + u * 32 + lane < nvec) {
                f32x2 x[NP];
                widen_pairs<DT>(raw[u], x);
#pragma unroll
                for (int j = 0; j < NP; ++j) { const f32x2 d = sub2(x[j], mu2); acc[j & 1] = fma2(d, d, acc[j & 1]); }
            }
        }
    }
    const float rstd = rstd_of(warp_sum<32>(pair_sum(add2(acc[0], acc[1]))) * inv_n, p.eps);
    const f32x2 r2 = pair(rstd, rstd);
    for (int k0 = 0; k0 < nvec; k0 += 32 * H) {
        uint4 raw[H], graw[H], braw[H];
#pragma unroll
        for (int u = 0; u < H; ++u) {
            const bool in = k0 + u * 32 + lane < nvec;
            raw[u] = make_uint4(0u, 0u, 0u, 0u); graw[u] = raw[u]; braw[u] = raw[u];
            if (in) raw[u] = sv[k0 + u * 32];
            if (gv && in) graw[u] = ld_cached(gv + k0 + u * 32);
            if (bv && in) braw[u] = ld_cached(bv + k0 + u * 32);
        }
#pragma unroll
        for (int u = 0; u < H; ++u) {
            if (k0 + u * 32 + lane < nvec) {
                f32x2 x[NP];
                widen_pairs<DT>(raw[u], x);
#pragma unroll
                for (int j = 0; j < NP; ++j) x[j] = sub2(x[j], mu2);
                affine_store_any<DT>(gv != nullptr, bv != nullptr, x, r2, graw[u], braw[u], yv + k0 + u * 32);
            }
        }
    }
}

// ---------------------------------------------------------------------------------------------
// cluster per row, slices resident in shared memory (one-shot grid: cluster i handles row i)
// dynamic shared memory: slice rounded up to whole chunks (stage_bytes) | 8 chunk mbarriers
// FULL: every block's slice is exactly nchunk_full chunks of 8 * blockDim.x vectors.
// ---------------------------------------------------------------------------------------------
constexpr int kNormMaxChunks = 8;

struct Pass2Ctx {
    const uint4* sv;       // this thread's first vector of the resident slice
    uint4* yv;             // and of the output row
    const uint4* gv;       // AFF 1: gamma / beta at the same column (null: absent)
    const uint4* bv;
    f32x2 mu2, r2;
    int nchunk, chunk_vecs, nv, tpos, v0;
};

// Pass 2 of the shared-memory kernel. Which affine vectors exist is a template parameter, chosen
// once per kernel: the loads of a half-chunk (x from shared memory, gamma and beta from L1/L2) are
// issued together, unconditionally, before any arithmetic.
template <int DT, bool FULL, int AFF, bool HG, bool HB>
__device__ __forceinline__ void norm_pass2(const NormParams& p, const Pass2Ctx& c, int64_t row) {
    constexpr int VE = Traits<DT>::VE;
    constexpr int NP = VE / 2;
    constexpr int H = 4;                                   // vectors per batch
    const int run_vecs = AFF == 2 ? static_cast<int>(p.run_elems / VE) : 1;
    const int64_t chan0 = AFF == 2 ? (row % p.aff_rows) * (p.nvec / run_vecs) : 0;     // first channel of this row's group
    for (int ch = 0; ch < c.nchunk; ++ch) {
#pragma unroll
        for (int half = 0; half < 2; ++half) {
            const int off = ch * c.chunk_vecs + half * H * 32;
            const int cbase = off + c.tpos;
            uint4 raw[H], graw[H], braw[H];
#pragma unroll
            for (int u = 0; u < H; ++u) raw[u] = c.sv[off + u * 32];
            if (AFF == 1) {
#pragma unroll
                for (int u = 0; u < H; ++u) {
                    const bool in = FULL || cbase + u * 32 < c.nv;      // never read past the end of gamma / beta
                    graw[u] = make_uint4(0u, 0u, 0u, 0u); braw[u] = make_uint4(0u, 0u, 0u, 0u);
                    if (HG && in) graw[u] = ld_cached(c.gv + off + u * 32);
                    if (HB && in) braw[u] = ld_cached(c.bv + off + u * 32);
                }
            }
#pragma unroll
            for (int u = 0; u < H; ++u) {
                if (FULL || cbase + u * 32 < c.nv) {
                    f32x2 x[NP];
                    widen_pairs<DT>(raw[u], x);
#pragma unroll
                    for (int k = 0; k < NP; ++k) x[k] = sub2(x[k], c.mu2);
                    if (AFF == 1) {
                        affine_store<DT, HG, HB>(x, c.r2, graw[u], braw[u], c.yv + off + u * 32);
                    } else if (AFF == 2) {
                        const int64_t chn = chan0 + (c.v0 + cbase + u * 32) / run_vecs;
                        const float gs = p.gamma ? load_elem<DT>(p.gamma, chn) : 1.0f;
                        const float bs = p.beta ? load_elem<DT>(p.beta, chn) : 0.0f;
                        float rlo, rhi;
                        unpair(c.r2, rlo, rhi);
                        const f32x2 a2 = pair(rlo * gs, rlo * gs), b2 = pair(bs, bs);
#pragma unroll
                        for (int k = 0; k < NP; ++k) x[k] = fma2(x[k], a2, b2);
                        st_stream(c.yv + off + u * 32, narrow_pairs<DT>(x));
                    } else {
                        affine_store<DT, false, false>(x, c.r2, raw[u], raw[u], c.yv + off + u * 32);
                    }
                }
            }
        }
    }
}

template <int DT, bool FULL, int AFF>
__global__ void __launch_bounds__(256, 3)
norm_smem_kernel(const NormParams p, const uint32_t stage_bytes, const int slice, const int nchunk_full) {
    constexpr int VE = Traits<DT>::VE;
    constexpr int NP = VE / 2;
    constexpr int U = 8;
    pdl_launch_dependents();
    extern __shared__ __align__(128) unsigned char smem[];
    __shared__ float4 wp[32];
    __shared__ __align__(16) float4 xchg[16];
    __shared__ __align__(8) uint64_t xbar;
    const int T = blockDim.x, tid = threadIdx.x, lane = tid & 31;
    const int tpos = (tid >> 5) * (32 * U) + lane;     // a warp owns 32 * U consecutive vectors of a chunk
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
    uint64_t* bars = reinterpret_cast<uint64_t*>(smem + stage_bytes);
    const uint4* sv = reinterpret_cast<const uint4*>(smem) + tpos;
    const int64_t row_bytes = p.nvec * 16;
    const char* xb = static_cast<const char*>(p.x) + int64_t(v0) * 16;

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
        if (cs > 1) mbar_expect_tx(smem_u32(&xbar), cs * 16u);
    }
    __syncthreads();
    if (cs > 1) {   // peers are resident, their mbarriers initialised, before any remote deposit
        cluster_arrive_relaxed();
        cluster_wait_acquire();
    }
    pdl_wait();

    // ---- pass 1: per chunk the exact (count, mean, M2) of this thread's vectors, merged as they land
    bool alive = true;
    Stat st = {0.0f, 0.0f, 0.0f};
    for (int ch = 0; ch < nchunk; ++ch) {
        if (tid < 32 && alive) alive = mbar_wait_warp(smem_u32(&bars[ch]), 0u, p.status);
        if (T > 32) __syncthreads();
        const uint4* sc = sv + ch * chunk_vecs;
        const int cbase = ch * chunk_vecs + tpos;
        uint4 raw[U];
        f32x2 acc[2] = {pair(0.0f, 0.0f), pair(0.0f, 0.0f)};
        int nvalid = U;
#pragma unroll
        for (int u = 0; u < U; ++u) {
            raw[u] = sc[u * 32];
            if (!FULL && cbase + u * 32 >= nv) { raw[u] = make_uint4(0u, 0u, 0u, 0u); --nvalid; }   // stale bytes past the slice
        }
#pragma unroll
        for (int u = 0; u < U; ++u) {
            f32x2 x[NP];
            widen_pairs<DT>(raw[u], x);
#pragma unroll
            for (int k = 0; k < NP; ++k) acc[k & 1] = add2(acc[k & 1], x[k]);
        }
        const float cnt = static_cast<float>(nvalid * VE);
        const float mean_c = nvalid > 0 ? pair_sum(add2(acc[0], acc[1])) * fast_rcp(cnt) : 0.0f;
        const f32x2 m2c = pair(mean_c, mean_c);
        acc[0] = pair(0.0f, 0.0f); acc[1] = pair(0.0f, 0.0f);
#pragma unroll
        for (int u = 0; u < U; ++u) {
            if (FULL || cbase + u * 32 < nv) {
                f32x2 x[NP];
                widen_pairs<DT>(raw[u], x);      // widened again rather than kept: 64 live values would not fit the register cap
#pragma unroll
                for (int k = 0; k < NP; ++k) {
                    const f32x2 d = sub2(x[k], m2c);
                    acc[k & 1] = fma2(d, d, acc[k & 1]);
                }
            }
        }
        Stat c;
        c.n = cnt; c.mean = mean_c; c.m2 = pair_sum(add2(acc[0], acc[1]));
        st = stat_merge(st, c);
    }
    // ---- merge: warp, block, cluster
    st = warp_merge_stats<32>(st);
    const int nwarps = T >> 5;
    if (nwarps > 1) {
        if (lane == 0) wp[tid >> 5] = make_float4(st.n, st.mean, st.m2, 0.0f);
        __syncthreads();
        const float4 v = lane < nwarps ? wp[lane] : make_float4(0.0f, 0.0f, 0.0f, 0.0f);
        st.n = v.x; st.mean = v.y; st.m2 = v.z;
        st = warp_merge_stats<32>(st);
    }
    if (cs > 1) {
        if (tid < cs) {
            const uint32_t dst = map_to_rank(smem_u32(&xchg[q]), tid), bar = map_to_rank(smem_u32(&xbar), tid);
            st_async_v2(dst, st.n, st.mean, bar);
            st_async_v2(dst + 8u, st.m2, 0.0f, bar);
        }
        cluster_arrive_relaxed();          // exit guard: waited for after pass 2 (see smem_row.cuh)
        if (tid < 32 && alive) alive = mbar_wait_warp(smem_u32(&xbar), 0u, p.status);
        if (T > 32) __syncthreads();
        const float4 v = lane < static_cast<int>(cs) ? xchg[lane] : make_float4(0.0f, 0.0f, 0.0f, 0.0f);
        st.n = v.x; st.mean = v.y; st.m2 = v.z;
        st = warp_merge_stats<32>(st);
    }
    const float rstd = rstd_of(st.m2 * fast_rcp(st.n), p.eps);
    const f32x2 mu2 = pair(st.mean, st.mean), r2 = pair(rstd, rstd);

    // ---- pass 2: normalise from the resident slice
    Pass2Ctx c2;
    c2.sv = sv; c2.yv = static_cast<uint4*>(p.y) + row * p.nvec + v0 + tpos;
    c2.gv = AFF == 1 && p.gamma ? static_cast<const uint4*>(p.gamma) + v0 + tpos : nullptr;
    c2.bv = AFF == 1 && p.beta ? static_cast<const uint4*>(p.beta) + v0 + tpos : nullptr;
    c2.mu2 = mu2; c2.r2 = r2; c2.nchunk = nchunk; c2.chunk_vecs = chunk_vecs; c2.nv = nv; c2.tpos = tpos; c2.v0 = v0;
    if (AFF == 1) {
        if (c2.gv && c2.bv) norm_pass2<DT, FULL, 1, true, true>(p, c2, row);
        else if (c2.gv)     norm_pass2<DT, FULL, 1, true, false>(p, c2, row);
        else                norm_pass2<DT, FULL, 1, false, true>(p, c2, row);
    } else {
        norm_pass2<DT, FULL, AFF, false, false>(p, c2, row);
    }
    if (cs > 1) cluster_wait_acquire();    // no block leaves while a peer's deposit into it is still to be issued
}

// ---------------------------------------------------------------------------------------------
// few, very long rows (group_norm of one large image): two kernels over a grid that fills the GPU.
//   norm_partial_kernel  block (row, b) takes segment b of the row (seg_vecs vectors), reduces it
//                        to one (n, mean, M2) triple and writes it to part[row * nseg + b]
//   norm_apply_kernel    the same grid: a block merges its row's nseg triples, then normalises its
//                        segment, re-reading x -- from L2 when the tensor fits there (the first
//                        kernel reads with the default policy, this one with evict-first)
// HBM traffic stays one read and one write per element when x fits L2; otherwise two reads.
// ---------------------------------------------------------------------------------------------
__device__ __forceinline__ uint4 ld_keep(const uint4* p) {
    FS_DBG_LOAD(p, 16, make_uint4(0u, 0u, 0u, 0u));
    uint4 v;
    asm volatile("ld.global.v4.u32 {%0,%1,%2,%3}, [%4];" : "=r"(v.x), "=r"(v.y), "=r"(v.z), "=r"(v.w) : "l"(p));
    return v;
}

// (n, mean, M2) of four vectors, exact two-pass in registers; absent vectors (valid < 4) are skipped.
template <int DT>
__device__ __forceinline__ Stat stat_of_vectors(const uint4 (&raw)[4], int valid) {
    constexpr int VE = Traits<DT>::VE;
    constexpr int NP = VE / 2;
    f32x2 acc[2] = {pair(0.0f, 0.0f), pair(0.0f, 0.0f)};
#pragma unroll
    for (int u = 0; u < 4; ++u) {
        f32x2 x[NP];
        widen_pairs<DT>(raw[u], x);                 // absent vectors were loaded as zeros
#pragma unroll
        for (int k = 0; k < NP; ++k) acc[k & 1] = add2(acc[k & 1], x[k]);
    }
    Stat c;
    c.n = static_cast<float>(valid * VE);
    c.mean = valid > 0 ? pair_sum(add2(acc[0], acc[1])) * fast_rcp(c.n) : 0.0f;
    const f32x2 m2 = pair(c.mean, c.mean);
    acc[0] = pair(0.0f, 0.0f); acc[1] = pair(0.0f, 0.0f);
#pragma unroll
    for (int u = 0; u < 4; ++u) {
        if (u < valid) {
            f32x2 x[NP];
            widen_pairs<DT>(raw[u], x);
#pragma unroll
            for (int k = 0; k < NP; ++k) { const f32x2 d = sub2(x[k], m2); acc[k & 1] = fma2(d, d, acc[k & 1]); }
        }
    }
    c.m2 = pair_sum(add2(acc[0], acc[1]));
    return c;
}

template <int DT>
__global__ void __launch_bounds__(256)
norm_partial_kernel(const NormParams p, float4* __restrict__ part, const int nseg, const int seg_vecs) {
    __shared__ float4 wp[32];
    pdl_launch_dependents();
    const int T = blockDim.x, tid = threadIdx.x, lane = tid & 31, nwarps = T >> 5;
    const int64_t row = blockIdx.x / nseg;
    const int b = static_cast<int>(blockIdx.x % nseg);
    const int64_t v0 = int64_t(b) * seg_vecs;
    const int nv = static_cast<int>(min(int64_t(seg_vecs), p.nvec - v0));
    const uint4* __restrict__ xv = static_cast<const uint4*>(p.x) + row * p.nvec + v0;
    pdl_wait();
    Stat st = {0.0f, 0.0f, 0.0f};
    for (int base = 0; base < nv; base += 4 * T) {          // a thread takes vectors base + tid + u T
        uint4 raw[4];
        int valid = 0;
#pragma unroll
        for (int u = 0; u < 4; ++u) {
            raw[u] = make_uint4(0u, 0u, 0u, 0u);
            if (base + tid + u * T < nv) { raw[u] = ld_keep(xv + base + tid + u * T); valid = u + 1; }
        }
        st = stat_merge(st, stat_of_vectors<DT>(raw, valid));
    }
    st = warp_merge_stats<32>(st);
    if (nwarps > 1) {
        if (lane == 0) wp[tid >> 5] = make_float4(st.n, st.mean, st.m2, 0.0f);
        __syncthreads();
        const float4 v = lane < nwarps ? wp[lane] : make_float4(0.0f, 0.0f, 0.0f, 0.0f);
        st.n = v.x; st.mean = v.y; st.m2 = v.z;
        st = warp_merge_stats<32>(st);
    }
    if (tid == 0) part[blockIdx.x] = make_float4(st.n, st.mean, st.m2, 0.0f);
}

template <int DT, int AFF>
__global__ void __launch_bounds__(256)
norm_apply_kernel(const NormParams p, const float4* __restrict__ part, const int nseg, const int seg_vecs) {
    constexpr int VE = Traits<DT>::VE;
    constexpr int NP = VE / 2;
    pdl_launch_dependents();
    const int T = blockDim.x, tid = threadIdx.x, lane = tid & 31;
    const int64_t row = blockIdx.x / nseg;
    const int b = static_cast<int>(blockIdx.x % nseg);
    const int64_t v0 = int64_t(b) * seg_vecs;
    const int nv = static_cast<int>(min(int64_t(seg_vecs), p.nvec - v0));
    const uint4* __restrict__ xv = static_cast<const uint4*>(p.x) + row * p.nvec + v0;
    uint4* __restrict__ yv = static_cast<uint4*>(p.y) + row * p.nvec + v0;
    pdl_wait();
    // every warp merges the row's partial triples (nseg <= 1024: up to 32 per lane)
    Stat st = {0.0f, 0.0f, 0.0f};
    for (int j = lane; j < nseg; j += 32) {
        const float4 v = part[row * nseg + j];
        Stat t; t.n = v.x; t.mean = v.y; t.m2 = v.z;
        st = stat_merge(st, t);
    }
    st = warp_merge_stats<32>(st);
    const float rstd = rstd_of(st.m2 * fast_rcp(st.n), p.eps);
    const f32x2 mu2 = pair(st.mean, st.mean), r2 = pair(rstd, rstd);
    const uint4* gv = AFF == 1 && p.gamma ? static_cast<const uint4*>(p.gamma) + v0 : nullptr;
    const uint4* bv = AFF == 1 && p.beta ? static_cast<const uint4*>(p.beta) + v0 : nullptr;
    const int run_vecs = AFF == 2 ? static_cast<int>(p.run_elems / VE) : 1;
    const int64_t chan0 = AFF == 2 ? (row % p.aff_rows) * (p.nvec / run_vecs) : 0;
    for (int base = 0; base < nv; base += 4 * T) {
        uint4 raw[4];
#pragma unroll
        for (int u = 0; u < 4; ++u) {
            raw[u] = make_uint4(0u, 0u, 0u, 0u);
            if (base + tid + u * T < nv) raw[u] = ld_stream(xv + base + tid + u * T);
        }
#pragma unroll
        for (int u = 0; u < 4; ++u) {
            const int v = base + tid + u * T;
            if (v < nv) {
                f32x2 x[NP];
                widen_pairs<DT>(raw[u], x);
#pragma unroll
                for (int k = 0; k < NP; ++k) x[k] = sub2(x[k], mu2);
                if (AFF == 1) {
                    uint4 graw = make_uint4(0u, 0u, 0u, 0u), braw = make_uint4(0u, 0u, 0u, 0u);
                    if (gv) graw = ld_cached(gv + v);
                    if (bv) braw = ld_cached(bv + v);
                    affine_store_any<DT>(gv != nullptr, bv != nullptr, x, r2, graw, braw, yv + v);
                } else if (AFF == 2) {
                    const int64_t chn = chan0 + (v0 + v) / run_vecs;
                    const float gs = p.gamma ? load_elem<DT>(p.gamma, chn) : 1.0f;
                    const float bs = p.beta ? load_elem<DT>(p.beta, chn) : 0.0f;
                    const f32x2 a2 = pair(rstd * gs, rstd * gs), b2 = pair(bs, bs);
#pragma unroll
                    for (int k = 0; k < NP; ++k) x[k] = fma2(x[k], a2, b2);
                    st_stream(yv + v, narrow_pairs<DT>(x));
                } else {
                    affine_store<DT, false, false>(x, r2, raw[u], raw[u], yv + v);
                }
            }
        }
    }
}

// ---------------------------------------------------------------------------------------------
// block per row, element-wise accesses, three passes (any shape and alignment)
// ---------------------------------------------------------------------------------------------
__device__ __forceinline__ float block_sum(float v, float* red) {
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5, nwarps = blockDim.x >> 5;
    v = warp_sum<32>(v);
    __syncthreads();                       // `red` may still be read from the previous reduction
    if (lane == 0) red[warp] = v;
    __syncthreads();
    v = lane < nwarps ? red[lane] : 0.0f;
    return warp_sum<32>(v);
}

template <int DT>
__global__ void __launch_bounds__(1024)
norm_generic_kernel(const NormParams p, const int aff) {
    __shared__ float red[32];
    pdl_launch_dependents();
    pdl_wait();
    const float inv_n = 1.0f / static_cast<float>(p.cols);
    for (int64_t row = blockIdx.x; row < p.rows; row += gridDim.x) {
        const int64_t base = row * p.cols;
        float s = 0.0f;
        for (int64_t j = threadIdx.x; j < p.cols; j += blockDim.x) s += load_elem<DT>(p.x, base + j);
        const float mu = block_sum(s, red) * inv_n;
        float q = 0.0f;
        for (int64_t j = threadIdx.x; j < p.cols; j += blockDim.x) {
            const float d = load_elem<DT>(p.x, base + j) - mu;
            q = fmaf(d, d, q);
        }
        const float rstd = rstd_of(block_sum(q, red) * inv_n, p.eps);
        const int64_t chan0 = aff == 2 ? (row % p.aff_rows) * (p.cols / p.run_elems) : 0;
        for (int64_t j = threadIdx.x; j < p.cols; j += blockDim.x) {
            float t = (load_elem<DT>(p.x, base + j) - mu) * rstd;
            if (aff) {
                const int64_t c = aff == 2 ? chan0 + j / p.run_elems : j;
                if (p.gamma) t *= load_elem<DT>(p.gamma, c);
                if (p.beta) t += load_elem<DT>(p.beta, c);
            }
            store_elem<DT>(p.y, base + j, t);
        }
    }
}

}  // namespace fsm
