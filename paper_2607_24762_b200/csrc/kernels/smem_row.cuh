// Split-row softmax with the slice resident in shared memory (long rows: vocabulary-sized, causal
// attention rows). A row is split over the CS blocks of a thread-block cluster (CS = 1: one block
// per row). Each block brings its slice into shared memory with bulk async copies, one mbarrier
// per chunk, and makes two passes over it:
//
//   pass 1  as the chunks land: every thread keeps a running (r, s) pair over its vectors, the
//           online-softmax update (Milakov-Gimelshein): a vector's own reference first, then
//           s <- s 2^((r - r')c) + sum 2^((x - r')c)
//   merge   warp shuffles -> block (one __syncthreads) -> cluster: each block deposits its pair
//           in every peer's shared memory with st.async, counted by an mbarrier there
//   pass 2  y = 2^((x - R)c) / S from the resident slice, 128-bit streaming stores
//
// Registers stay low (no per-thread copy of the row), so occupancy is set by shared memory:
// several blocks per SM in different phases keep HBM busy. Cost: two ex2 per element.
#pragma once
#include "block_row.cuh"
#include "common.cuh"

namespace fsm {

constexpr int kSmemRowMaxChunks = 16;

// Dynamic shared memory: slice (stage_bytes) | kSmemRowMaxChunks chunk mbarriers.
// chunk_vecs is a multiple of blockDim.x.
template <int DT, bool NEG>
__global__ void __launch_bounds__(512, 2)
smem_row_kernel(const Params p, const uint32_t stage_bytes, const int slice, const int chunk_vecs) {
    constexpr int VE = Traits<DT>::VE;
    constexpr int U = 4;                                  // vectors a thread handles per step
    pdl_launch_dependents();
    extern __shared__ __align__(128) unsigned char smem[];
    __shared__ float2 wp[2][32];
    __shared__ __align__(16) float2 xchg[2][16];
    __shared__ __align__(8) uint64_t xbar[2];
    const int T = blockDim.x, tid = threadIdx.x, lane = tid & 31;
    const uint32_t q = cluster_ctarank(), cs = cluster_nctarank();
    const int64_t ncl = cluster_count_x();
    const int64_t cid = cluster_id_x();
    const int nvec = static_cast<int>(p.nvec);
    const int v0 = min(nvec, static_cast<int>(q) * slice);
    const int nv = min(nvec, v0 + slice) - v0;            // vectors of this block's slice (may be 0)
    const int nchunk = (nv + chunk_vecs - 1) / chunk_vecs;
    const float ident = ref_identity<NEG>();
    uint64_t* bars = reinterpret_cast<uint64_t*>(smem + stage_bytes);
    const uint4* sv = reinterpret_cast<const uint4*>(smem);
    const char* xb = static_cast<const char*>(p.x);
    uint4* __restrict__ yv = static_cast<uint4*>(p.y);
    const int64_t row_bytes = p.nvec * 16;
    const int64_t n_my = cid < p.rows ? (p.rows - cid + ncl - 1) / ncl : 0;   // same for the whole cluster

    auto issue_row = [&](int64_t row) {                    // thread 0: one bulk copy per chunk
        for (int ch = 0; ch < nchunk; ++ch) {
            const int cv = min(chunk_vecs, nv - ch * chunk_vecs);
            bulk_load_row(smem_u32(smem) + uint32_t(ch) * uint32_t(chunk_vecs) * 16u,
                          xb + row * row_bytes + (int64_t(v0) + int64_t(ch) * chunk_vecs) * 16,
                          uint32_t(cv) * 16u, smem_u32(&bars[ch]));
        }
    };

    if (tid == 0) {
        for (int ch = 0; ch < kSmemRowMaxChunks; ++ch) mbar_init(smem_u32(&bars[ch]), 1);
        mbar_init(smem_u32(&xbar[0]), 1);
        mbar_init(smem_u32(&xbar[1]), 1);
        mbar_fence_init();
        fence_proxy_async_smem();
        pdl_wait();
        if (n_my > 0) issue_row(cid);
    }
    __syncthreads();
    if (cs > 1) {   // peers are resident, their mbarriers initialised, before any remote deposit
        cluster_arrive_relaxed();
        cluster_wait_acquire();
    }
    pdl_wait();

    bool alive = true;      // false once a bounded wait has expired: later waits are skipped
    for (int64_t i = 0; i < n_my; ++i) {
        const int64_t row = cid + i * ncl;
        const int par = static_cast<int>(i & 1);
        const uint32_t phase = static_cast<uint32_t>(i) & 1u;
        if (cs > 1 && tid == 0) mbar_expect_tx(smem_u32(&xbar[par]), cs * 8u);

        // ---- pass 1: running (r, s) over this thread's vectors, chunk by chunk as they land.
        // A chunk gives a thread U vectors: their common reference first, one rescale of s, then
        // one ex2 per element.
        float r = ident, s = 0.0f;
        for (int ch = 0; ch < nchunk; ++ch) {
            if (alive) alive = mbar_wait_warp(smem_u32(&bars[ch]), phase, p.status);
            const int cbeg = ch * chunk_vecs, cend = min(nv, cbeg + chunk_vecs);
            for (int v0c = cbeg + tid; v0c < cend; v0c += U * T) {
                uint4 raw[U];
                RefAcc<DT, NEG> acc;
                acc.init();
#pragma unroll
                for (int u = 0; u < U; ++u) {
                    raw[u] = make_uint4(0u, 0u, 0u, 0u);
                    if (v0c + u * T < cend) { raw[u] = sv[v0c + u * T]; acc.fold(raw[u]); }
                }
                const float rn = ref_pick<NEG>(r, acc.value());
                if (rn != r) { s *= ref_factor(r, rn, p.c, ident); r = rn; }
                const float ru = (rn == ident) ? 0.0f : rn;
                float part = 0.0f;
#pragma unroll
                for (int u = 0; u < U; ++u) {
                    if (v0c + u * T < cend) {
                        float e[VE];
                        unpack<DT>(raw[u], e);
#pragma unroll
                        for (int k = 0; k < VE; ++k) part += ex2_elem<DT>(e[k] - ru, p.c);
                    }
                }
                s += part;
            }
        }
        float R = r;
        block_merge_pairs<NEG>(R, s, wp[par], p.c);
        if (cs > 1) {
            if (tid < cs)
                st_async_v2(map_to_rank(smem_u32(&xchg[par][q]), tid), R, s, map_to_rank(smem_u32(&xbar[par]), tid));
            if (alive) alive = mbar_wait_warp(smem_u32(&xbar[par]), static_cast<uint32_t>(i >> 1) & 1u, p.status);
            R = ident; s = 0.0f;
            if (lane < static_cast<int>(cs)) ld_shared_v2(smem_u32(&xchg[par][lane]), R, s);
            warp_merge_pairs<NEG>(R, s, p.c);
        }

        // ---- pass 2: normalise from the resident slice
        const float inv = recip<DT>(s);
        const float Ru = (R == ident) ? 0.0f : R;
        uint4* yrow = yv + row * p.nvec + v0;
        for (int vb = tid; vb < nv; vb += U * T) {
            uint4 raw[U];
#pragma unroll
            for (int u = 0; u < U; ++u)
                if (vb + u * T < nv) raw[u] = sv[vb + u * T];
#pragma unroll
            for (int u = 0; u < U; ++u) {
                if (vb + u * T < nv) {
                    float e[VE];
                    unpack<DT>(raw[u], e);
#pragma unroll
                    for (int k = 0; k < VE; ++k) e[k] = ex2_elem<DT>(e[k] - Ru, p.c) * inv;
                    st_stream(yrow + vb + u * T, pack<DT>(e));
                }
            }
        }

        if (i + 1 < n_my) {     // resident-grid form: the slice is free once everyone has read it
            __syncthreads();
            if (tid == 0) { fence_proxy_async_smem(); issue_row(row + ncl); }
        }
    }
}

}  // namespace fsm
