// softmax(scale * x + mask) with the addition done in the kernel: eager attention forms
// `scores + mask` as a tensor of its own before the softmax (one more read and write of the
// scores); here the mask row is read beside the score row -- it is shared by all heads, so it
// stays in L2 -- and the sum never exists in memory.
//
// Base-2 exponent of element j:  t_j = x_j * c + m_j * log2(e)   (one fused multiply-add; c = scale
// * log2 e), reference R = max_j t_j, e_j = 2^(t_j - R). Unlike the plain kernels the product
// x_j * c is formed before the reference is subtracted (the mask makes the reference depend on
// both terms), so the exponent carries the binary32 rounding of a number of the size of |z|: the
// parity bound of this entry point grows with max |z| (see the header).
//
//   sm_masked_warp_kernel     (sub-)warp per row, the row packed in registers (rows up to 9 KiB)
//   sm_masked_tile_kernel     rows of 4-11 KiB: four rows per block in shared memory, a warp per row
//   sm_masked_smem_kernel     the split-row design: x slice resident in shared memory, mask slice
//                             read from L2 in pass 1 only (e is stored in place, as in smem_row)
//   sm_masked_generic_kernel  block per row, element-wise, any shape and alignment
#pragma once
#include "block_row.cuh"
#include "common.cuh"
#include "norm_row.cuh"

namespace fsm {

struct MaskedParams {
    const void* x;
    const void* mask;
    void* y;
    int64_t rows;
    int64_t cols;
    int64_t nvec;
    int64_t q_rows;      // mask row of row i: (i / (heads * q_rows)) * q_rows + i % q_rows
    int64_t group;       // heads * q_rows
    float c;             // scale * log2(e)
    int* status;
    int64_t pf_rows;
    float lag_ns;          // first wave of a one-shot grid: cluster i < lag_rows starts i * lag_ns late
    int lag_rows;
    int early_pf;          // first wave: ask L2 for the block's own input before griddepcontrol.wait (pdl_early_prefetch)
};

__device__ __forceinline__ int64_t mask_row_of(const MaskedParams& p, int64_t row) {
    return (row / p.group) * p.q_rows + row % p.q_rows;
}

constexpr float kLog2eF = 1.4426950408889634f;

// t = x * c + m * log2(e) for one vector, as pairs; returns the largest t (NaN dropped, like fmaxf).
template <int DT>
__device__ __forceinline__ float masked_exponents(const uint4& xraw, const uint4& mraw, f32x2 c2, f32x2 (&t)[Traits<DT>::VE / 2]) {
    constexpr int NP = Traits<DT>::VE / 2;
    f32x2 m[NP];
    widen_pairs<DT>(xraw, t);
    widen_pairs<DT>(mraw, m);
    const f32x2 l2 = pair(kLog2eF, kLog2eF);
    float best = __int_as_float(0xff800000);
#pragma unroll
    for (int k = 0; k < NP; ++k) {
        t[k] = fma2(t[k], c2, mul2(m[k], l2));
        float lo, hi;
        unpair(t[k], lo, hi);
        best = fmaxf(best, fmaxf(lo, hi));
    }
    return best;
}

// ---------------------------------------------------------------------------------------------
// The row stays packed in registers; the mask vectors are not kept but read twice through the
// read-only path (they are shared by the heads and hit L1/L2). Pass A takes the maximum exponent,
// pass B forms e = 2^(t - R), adds it up and puts it back in place of x in the element dtype
// (the in-place store of the split-row kernel, in registers), pass C scales and stores.
// The single sweep of sm_masked_tile_kernel below (exponents formed once, per-batch references) was
// tried here too and is slower: holding a batch's 32 exponents takes 72 registers against 56 and the
// resident warps are what hides the latency of this kernel (bf16 rows of 1 / 2 / 3 KiB: 10.1 -> 11.2,
// 16.5 -> 18.4, 23.5 -> 27.5 us; fp32 rows of 4 KiB 23.2 -> 24.2 us).
template <int DT, int LANES, int VPL>
__device__ __forceinline__ void sm_masked_warp_body(const MaskedParams& p) {
    constexpr int NP = Traits<DT>::VE / 2;
    constexpr int G = 32 / LANES;
    pdl_launch_dependents();
    const int lane = threadIdx.x & 31;
    const int sub = lane / LANES, sl = lane % LANES;
    const int warps = blockDim.x >> 5;
    const int nvec = static_cast<int>(p.nvec);
    const uint4* __restrict__ xv = static_cast<const uint4*>(p.x);
    const uint4* __restrict__ mv = static_cast<const uint4*>(p.mask);
    uint4* __restrict__ yv = static_cast<uint4*>(p.y);
    const f32x2 c2 = pair(p.c, p.c);
    pdl_wait();
    const int64_t ngroups = (p.rows + G - 1) / G;
    for (int64_t grp = int64_t(blockIdx.x) * warps + (threadIdx.x >> 5); grp < ngroups; grp += int64_t(gridDim.x) * warps) {
        const int64_t row = grp * G + sub;
        const bool row_ok = row < p.rows;
        const uint4* mr = mv + (row_ok ? mask_row_of(p, row) : 0) * p.nvec + sl;
        uint4 xraw[VPL];
#pragma unroll
        for (int k = 0; k < VPL; ++k) {
            xraw[k] = make_uint4(0u, 0u, 0u, 0u);
            if (row_ok && sl + k * LANES < nvec) xraw[k] = ld_stream(xv + row * p.nvec + sl + k * LANES);
        }
        float r = __int_as_float(0xff800000);
#pragma unroll
        for (int k = 0; k < VPL; ++k) {
            if (row_ok && sl + k * LANES < nvec) {
                f32x2 t[NP];
                r = fmaxf(r, masked_exponents<DT>(xraw[k], ld_cached(mr + k * LANES), c2, t));
            }
        }
        r = warp_pick<LANES, false>(r);
        const f32x2 r2 = pair(r, r);
        f32x2 acc[2] = {pair(0.0f, 0.0f), pair(0.0f, 0.0f)};
#pragma unroll
        for (int k = 0; k < VPL; ++k) {
            if (row_ok && sl + k * LANES < nvec) {
                f32x2 t[NP];
                masked_exponents<DT>(xraw[k], ld_cached(mr + k * LANES), c2, t);
#pragma unroll
                for (int j = 0; j < NP; ++j) {
                    float lo, hi;
                    unpair(sub2(t[j], r2), lo, hi);
                    if (DT == DT_BF16) { lo += 64.0f; hi += 64.0f; }        // keeps subnormal bf16 outputs (see ex2_elem)
                    t[j] = pair(ex2_ftz(lo), ex2_ftz(hi));
                    acc[j & 1] = add2(acc[j & 1], t[j]);
                }
                xraw[k] = narrow_pairs<DT>(t);
            }
        }
        const float inv = recip<DT>(warp_sum<LANES>(pair_sum(add2(acc[0], acc[1]))));
        const f32x2 i2 = pair(inv, inv);
        if (row_ok) {
#pragma unroll
            for (int k = 0; k < VPL; ++k)
                if (sl + k * LANES < nvec) st_stream(yv + row * p.nvec + sl + k * LANES, scale_vec<DT, false>(xraw[k], i2, i2));
        }
    }
}

// Up to eight vectors per lane the compiler's own register choice is best (an explicit minimum of
// blocks per SM, even 1, makes it spend registers: measured 88 us against 80 on short rows); the
// long-row variants are capped so that four or five blocks stay resident.
template <int DT, int LANES, int VPL>
__global__ void __launch_bounds__(128)
sm_masked_warp_kernel(const MaskedParams p) {
    sm_masked_warp_body<DT, LANES, VPL>(p);
}
template <int DT, int VPL>
__global__ void __launch_bounds__(128, VPL <= 12 ? 5 : 4)
sm_masked_warp_long_kernel(const MaskedParams p) {
    sm_masked_warp_body<DT, 32, VPL>(p);
}

// ---------------------------------------------------------------------------------------------
// 16-bit rows of 4-10 KiB: four rows per block, each brought to shared memory by a bulk copy of its
// own (one mbarrier per row) and worked on by one warp alone, in NB batches of 4 vectors per lane.
// The exponents t = x c + m log2(e) are formed ONCE (the mask vectors are read once, through the
// read-only path): a lane takes the largest t of its 32 elements of the batch as that batch's
// reference r_b, puts e = 2^(t - r_b) back in place of x in shared memory in the element dtype and
// folds the batch's sum into its running (r, s) pair with the online-softmax merge
// (Milakov-Gimelshein); the lanes' pairs are merged by shuffles, and the last sweep stores
// y = e * 2^(r_b - R) / S, the per-batch factor being one ex2 per lane and batch. This is the
// split-row kernel's arithmetic (smem_row.cuh: chunk references, in-place e, the bf16 bias of 2^64
// and the separate small factor) with a lane's batch in the role of a thread's chunk; the bias is
// folded into the reference (r_b - 64 is what is subtracted and what is merged), which saves the
// addition per element. A first version took the row maximum in a sweep of its own and formed t
// twice: 21.5 thread instructions per element and 27.9 us on 8 x 2048 rows of 4 KiB bf16 with a
// shared mask, issue-bound; this one takes 23.4 us (rows of 5 / 8 / 10 KiB: 35.5 -> 31.8, 33.7 -> 26.7, 41.8 -> 32.9 us).
// FULL: the row is exactly NB batches (no bounds checks). No block barrier after start-up.
// One-shot grid: block b handles rows b*W .. b*W+W-1. dynamic shared memory: W rows | W mbarriers
// ---------------------------------------------------------------------------------------------
template <int DT, int NB, bool FULL>
__global__ void __launch_bounds__(128)
sm_masked_tile_kernel(const MaskedParams p) {
    static_assert(DT != DT_F32, "16-bit element types only");
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
    uint4* sv = reinterpret_cast<uint4*>(smem + size_t(w) * size_t(row_bytes)) + lane;
    const uint4* __restrict__ mr = static_cast<const uint4*>(p.mask) + mask_row_of(p, row) * p.nvec + lane;
    uint4* __restrict__ yv = static_cast<uint4*>(p.y) + row * p.nvec + lane;
    const f32x2 c2 = pair(p.c, p.c);
    const float ident = __int_as_float(0xff800000);
    const uint32_t ninf = DT == DT_BF16 ? 0xff80ff80u : 0xfc00fc00u;     // a vector past the row's end: x = 0, mask = -inf
    mbar_wait_warp(smem_u32(&bars[w]), 0u, p.status);      // on a timeout the status word is set and the row is garbage

    float rb[NB];                                          // what batch b's e are relative to (ident: nothing but -inf or NaN)
    float r = ident, s = 0.0f;
#pragma unroll
    for (int b = 0; b < NB; ++b) {
        const int k0 = b * 32 * H;
        uint4 xr[H], mk[H];
#pragma unroll
        for (int u = 0; u < H; ++u) {
            xr[u] = make_uint4(0u, 0u, 0u, 0u); mk[u] = make_uint4(ninf, ninf, ninf, ninf);
            if (FULL || k0 + u * 32 + lane < nvec) { xr[u] = sv[k0 + u * 32]; mk[u] = ld_cached(mr + k0 + u * 32); }
        }
        f32x2 t[H][NP];
        float m = ident;
#pragma unroll
        for (int u = 0; u < H; ++u) m = fmaxf(m, masked_exponents<DT>(xr[u], mk[u], c2, t[u]));
        // all of these elements masked (or none finite): subtract 0 instead of the identity. bf16: e carries
        // 2^64 so that outputs below 2^-126 survive in e (see ex2_elem); the bias sits in the reference.
        const float sub = ((m == ident) ? 0.0f : m) - (DT == DT_BF16 ? 64.0f : 0.0f);
        rb[b] = (m == ident) ? ident : sub;
        const f32x2 s2 = pair(sub, sub);
        f32x2 acc[2] = {pair(0.0f, 0.0f), pair(0.0f, 0.0f)};
#pragma unroll
        for (int u = 0; u < H; ++u) {
#pragma unroll
            for (int j = 0; j < NP; ++j) {
                float lo, hi;
                unpair(sub2(t[u][j], s2), lo, hi);
                t[u][j] = pair(ex2_ftz(lo), ex2_ftz(hi));
                acc[j & 1] = add2(acc[j & 1], t[u][j]);
            }
            if (FULL || k0 + u * 32 + lane < nvec) sv[k0 + u * 32] = narrow_pairs<DT>(t[u]);     // this lane alone reads it back
        }
        const float part = pair_sum(add2(acc[0], acc[1]));
        // online merge of (rb[b], part) into (r, s): only the sum left behind is rescaled
        const float rn = fmaxf(r, rb[b]);
        const bool keep = (rn == r);
        const float lo = keep ? rb[b] : r;
        const float f = (lo == ident) ? 1.0f : ex2_ftz(lo - rn);
        s = keep ? fmaf(part, f, s) : fmaf(s, f, part);
        r = rn;
    }
    warp_merge_pairs<false>(r, s, 1.0f);
    const float inv = recip<DT>(s);
#pragma unroll
    for (int b = 0; b < NB; ++b) {
        const int k0 = b * 32 * H;
        const float fac = (rb[b] == ident) ? 1.0f : ex2_noflush(rb[b] - r);
        // bf16: e carries 2^64 and inv 2^-64; a factor this small is applied separately so that
        // fac * inv cannot underflow before it meets e
        const bool one_mul = DT != DT_BF16 || fac >= 0x1p-40f || !(fac == fac);
        const float f1 = one_mul ? fac * inv : inv;
        const f32x2 f2 = pair(f1, f1), g2 = pair(fac, fac);
        uint4 e[H];
#pragma unroll
        for (int u = 0; u < H; ++u) {
            e[u] = make_uint4(0u, 0u, 0u, 0u);
            if (FULL || k0 + u * 32 + lane < nvec) e[u] = sv[k0 + u * 32];
        }
        if (one_mul) {
#pragma unroll
            for (int u = 0; u < H; ++u)
                if (FULL || k0 + u * 32 + lane < nvec) st_stream(yv + k0 + u * 32, scale_vec<DT, false>(e[u], f2, f2));
        } else {                                           // rare: both multiplications before the one rounding
#pragma unroll
            for (int u = 0; u < H; ++u)
                if (FULL || k0 + u * 32 + lane < nvec) st_stream(yv + k0 + u * 32, scale_vec<DT, true>(e[u], f2, g2));
        }
    }
}

// ---------------------------------------------------------------------------------------------
// cluster per row (one-shot grid); dynamic shared memory: x slice rounded up to whole chunks
// (stage_bytes) | 8 chunk mbarriers | per-thread chunk references (8 * blockDim.x floats)
// ---------------------------------------------------------------------------------------------
template <int DT, bool FULL>
__global__ void __launch_bounds__(256, 3)
sm_masked_smem_kernel(const MaskedParams p, const uint32_t stage_bytes, const int slice, const int nchunk_full) {
    constexpr int VE = Traits<DT>::VE;
    constexpr int NP = VE / 2;
    constexpr int U = 8;
    pdl_launch_dependents();
    extern __shared__ __align__(128) unsigned char smem[];
    __shared__ float2 wp[32];
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
    float* rcs = reinterpret_cast<float*>(smem + stage_bytes + kNormMaxChunks * 8) + tid;       // [chunk][thread]
    uint4* sv = reinterpret_cast<uint4*>(smem) + tpos;
    const int64_t row_bytes = p.nvec * 16;
    const char* xb = static_cast<const char*>(p.x) + int64_t(v0) * 16;
    const uint4* mv = static_cast<const uint4*>(p.mask) + mask_row_of(p, row) * p.nvec + v0 + tpos;
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

    // ---- pass 1: exponents of a half-chunk at a time, its reference, e stored in place
    bool alive = true;
    float r = ident, s = 0.0f;
    for (int ch = 0; ch < nchunk; ++ch) {
        // the mask vectors of the chunk are requested before the wait for the chunk's x
        uint4 mraw[U];
        const int cbase = ch * chunk_vecs + tpos;
#pragma unroll
        for (int u = 0; u < U; ++u) {
            mraw[u] = make_uint4(0u, 0u, 0u, 0u);
            if (FULL || cbase + u * 32 < nv) mraw[u] = ld_cached(mv + ch * chunk_vecs + u * 32);
        }
        if (tid < 32 && alive) alive = mbar_wait_warp(smem_u32(&bars[ch]), 0u, p.status);
        if (T > 32) __syncthreads();
        uint4* sc = sv + ch * chunk_vecs;
        float rch[2];
        float part[2];
#pragma unroll
        for (int h = 0; h < 2; ++h) {
            f32x2 t[U / 2][NP];
            float rc = ident;
#pragma unroll
            for (int u = 0; u < U / 2; ++u) {
                const int uu = h * (U / 2) + u;
                const float b = masked_exponents<DT>(sc[uu * 32], mraw[uu], c2, t[u]);
                if (FULL || cbase + uu * 32 < nv) rc = fmaxf(rc, b);
            }
            const float ru = (rc == ident) ? 0.0f : rc;
            const f32x2 ru2 = pair(ru, ru);
            f32x2 acc[2] = {pair(0.0f, 0.0f), pair(0.0f, 0.0f)};
#pragma unroll
            for (int u = 0; u < U / 2; ++u) {
                const int uu = h * (U / 2) + u;
                if (FULL || cbase + uu * 32 < nv) {
#pragma unroll
                    for (int k = 0; k < NP; ++k) {
                        float lo, hi;
                        unpair(sub2(t[u][k], ru2), lo, hi);
                        if (DT == DT_BF16) { lo += 64.0f; hi += 64.0f; }
                        t[u][k] = pair(ex2_ftz(lo), ex2_ftz(hi));
                        acc[k & 1] = add2(acc[k & 1], t[u][k]);
                    }
                    sc[uu * 32] = narrow_pairs<DT>(t[u]);
                }
            }
            rch[h] = rc;
            part[h] = pair_sum(add2(acc[0], acc[1]));
        }
        // the two halves have their own references: fold the second into the first, keep both for pass 2
        rcs[(2 * ch) * T] = rch[0];
        rcs[(2 * ch + 1) * T] = rch[1];
#pragma unroll
        for (int h = 0; h < 2; ++h) {
            const float rc = rch[h];
            const float rn = fmaxf(r, rc);
            const bool keep = (rn == r);
            const float lo = keep ? rc : r;
            const float f = (lo == ident) ? 1.0f : ex2_ftz((lo - rn));
            s = keep ? fmaf(part[h], f, s) : fmaf(s, f, part[h]);
            r = rn;
        }
    }
    // (r, s) pairs here are in base-2 exponent units already: merge with c = 1
    float R = r;
    block_merge_pairs<false>(R, s, wp, 1.0f);
    if (cs > 1) {
        if (tid < cs) st_async_v2(map_to_rank(smem_u32(&xchg[q]), tid), R, s, map_to_rank(smem_u32(&xbar), tid));
        cluster_arrive_relaxed();          // exit guard: waited for after pass 2 (see smem_row.cuh)
        if (tid < 32 && alive) alive = mbar_wait_warp(smem_u32(&xbar), 0u, p.status);
        if (T > 32) __syncthreads();
        R = ident; s = 0.0f;
        if (lane < static_cast<int>(cs)) ld_shared_v2(smem_u32(&xchg[lane]), R, s);
        warp_merge_pairs<false>(R, s, 1.0f);
    }

    // ---- pass 2: scale the stored e, half-chunk by half-chunk with its own reference
    const float inv = recip<DT>(s);
    uint4* __restrict__ yv = static_cast<uint4*>(p.y) + row * p.nvec + v0 + tpos;
    for (int ch = 0; ch < nchunk; ++ch) {
        const uint4* sc = sv + ch * chunk_vecs;
        const int cbase = ch * chunk_vecs + tpos;
#pragma unroll
        for (int h = 0; h < 2; ++h) {
            const float rc = rcs[(2 * ch + h) * T];
            const float fac = (rc == ident) ? 1.0f : ex2_noflush(rc - R);
            const bool one_mul = DT != DT_BF16 || fac >= 0x1p-40f || !(fac == fac);
            const float f1 = one_mul ? fac * inv : inv;
            const f32x2 f2 = pair(f1, f1), g2 = pair(fac, fac);
            uint4 raw[U / 2];
#pragma unroll
            for (int u = 0; u < U / 2; ++u) raw[u] = sc[(h * (U / 2) + u) * 32];
            if (DT == DT_BF16 && !one_mul) {
#pragma unroll
                for (int u = 0; u < U / 2; ++u) {
                    const int uu = h * (U / 2) + u;
                    if (FULL || cbase + uu * 32 < nv) st_stream(yv + ch * chunk_vecs + uu * 32, scale_vec<DT, true>(raw[u], f2, g2));
                }
            } else {
#pragma unroll
                for (int u = 0; u < U / 2; ++u) {
                    const int uu = h * (U / 2) + u;
                    if (FULL || cbase + uu * 32 < nv) st_stream(yv + ch * chunk_vecs + uu * 32, scale_vec<DT, false>(raw[u], f2, f2));
                }
            }
        }
    }
    if (cs > 1) cluster_wait_acquire();    // no block leaves while a peer's deposit into it is still to be issued
}

// ---------------------------------------------------------------------------------------------
template <int DT>
__global__ void __launch_bounds__(1024)
sm_masked_generic_kernel(const MaskedParams p) {
    __shared__ float red[32];
    pdl_launch_dependents();
    pdl_wait();
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5, nwarps = blockDim.x >> 5;
    for (int64_t row = blockIdx.x; row < p.rows; row += gridDim.x) {
        const int64_t base = row * p.cols, mbase = mask_row_of(p, row) * p.cols;
        float m = ref_identity<false>();
        for (int64_t j = threadIdx.x; j < p.cols; j += blockDim.x)
            m = fmaxf(m, fmaf(load_elem<DT>(p.x, base + j), p.c, load_elem<DT>(p.mask, mbase + j) * kLog2eF));
        m = warp_pick<32, false>(m);
        __syncthreads();
        if (lane == 0) red[warp] = m;
        __syncthreads();
        m = warp_pick<32, false>(lane < nwarps ? red[lane] : ref_identity<false>());
        float s = 0.0f;
        for (int64_t j = threadIdx.x; j < p.cols; j += blockDim.x)
            s += ex2_noflush(fmaf(load_elem<DT>(p.x, base + j), p.c, load_elem<DT>(p.mask, mbase + j) * kLog2eF) - m);
        const float inv = 1.0f / block_sum(s, red);
        for (int64_t j = threadIdx.x; j < p.cols; j += blockDim.x)
            store_elem<DT>(p.y, base + j,
                           ex2_noflush(fmaf(load_elem<DT>(p.x, base + j), p.c, load_elem<DT>(p.mask, mbase + j) * kLog2eF) - m) * inv);
    }
}

}  // namespace fsm
