// Split-row softmax with the slice resident in shared memory (long rows: vocabulary-sized, causal
// attention rows). A row is split over the CS blocks of a thread-block cluster (CS = 1: one block
// per row; any size up to 16). Each block brings its slice into shared memory with bulk async
// copies, one mbarrier per chunk (a chunk = eight vectors per thread), and makes two passes over it:
//
//   pass 1  as the chunks land: a thread takes its eight vectors of the chunk, their reference r_c
//           first (packed max), then e = 2^((x - r_c)c) for every element: one ex2 per element,
//           the subtraction, the scaling and the summation two elements per instruction
//           (f32x2). The e are added (fp32, unrounded) to the thread's running (r, s) pair with
//           the online-softmax merge (Milakov-Gimelshein), and written back IN PLACE over x in
//           the element's own dtype; r_c goes to a small per-thread table in shared memory.
//   merge   warp shuffles -> block (one __syncthreads) -> cluster: each block deposits its pair
//           in every peer's shared memory with st.async, counted by an mbarrier there
//   pass 2  y = e * 2^((r_c - R)c) / S from the resident slice: no second ex2 per element
//
// Within a chunk a warp owns 32 * 8 consecutive vectors and a lane every 32nd of them, so the
// offsets of a thread's eight vectors are compile-time constants (no address arithmetic per
// access) while every warp-wide access stays contiguous.
//
// Storing e rounded to the output dtype keeps the result within the stated bar: for fp32 it is
// exact; for bf16/fp16 it moves e, hence the unrounded y, by less than one unit in the last place
// of y (half a unit of e is at most one unit of y = e * f), and two values less than one unit
// apart round to the same or to adjacent numbers (the row sum is taken over the unrounded e).
//
// Registers stay low (no per-thread copy of the row), so occupancy is set by shared memory:
// several blocks per SM in different phases keep HBM busy, and thread 0 asks L2 for the slice of a
// row that starts a fraction of a generation later, so that DRAM reads do not stop while the
// resident blocks compute.
#pragma once
#include "block_row.cuh"
#include "common.cuh"

namespace fsm {

constexpr int kSmemRowMaxChunks = 8;
// Vectors a thread takes from a chunk: 8 (32 fp32 or 64 16-bit elements per step). With blocks of
// at most 256 threads and a cap of 85 registers, three 256-thread or six 128-thread blocks fit an SM.
__host__ __device__ constexpr int smem_row_u(int) { return 8; }
// What follows the slice in dynamic shared memory: kSmemRowMaxChunks chunk mbarriers, then one
// reference per (chunk, thread) for the chunks the geometry really has.
constexpr uint32_t kSmemRowBarBytes = kSmemRowMaxChunks * 8;
__host__ __device__ constexpr uint32_t smem_row_tail_bytes(int threads, int nchunk) {
    return kSmemRowBarBytes + uint32_t(nchunk) * uint32_t(threads) * 4u;
}

// Dynamic shared memory: slice rounded up to whole chunks (stage_bytes = nchunk_alloc chunks) |
// kSmemRowMaxChunks chunk mbarriers | per-thread chunk references (nchunk_alloc * blockDim.x floats).
// The slice must fit in kSmemRowMaxChunks chunks of smem_row_u(DT) * blockDim.x vectors.
//
// Who waits for a chunk. Thread 0 issues one bulk copy per chunk; warp 0 polls the chunk's mbarrier
// (one lane, spaced by nanosleep) and the other warps wait for warp 0 at the block's hardware
// barrier, where a waiting warp costs no issue slot. Measured on B200 (256 rows of 512 KiB bf16)
// against the alternative that needs no block barrier in the chunk loop -- every warp owning a
// contiguous 4 KiB range of each chunk, with its own copy and its own mbarrier, and waiting for the
// cluster's exchange barrier by itself: 49.9 us against 47.1. The profiler shows why: 19% more warp
// instructions (27.1 M against 22.8 M), all of them polls; a polling lane is a warp instruction
// every few hundred nanoseconds in each of four warps instead of one, on SMs whose issue slots are
// half used by the arithmetic of the other resident blocks.
//
// FULL: every block's slice is exactly nchunk_alloc chunks (no per-vector bounds checks, no
// integer division in the prologue).
// Rows cid, cid + clusters, ... are handled by cluster cid (normally exactly one row).
// CAUSAL (one cluster per row, not FULL): row i keeps its first min(cols, i + q_offset + 1)
// columns; only those are fetched, the vector that straddles the boundary gets its masked lanes
// replaced by the reference identity, and the rest of the row is filled with 0 * (1/S): +0, or NaN
// for a row that is NaN or has no column left.
//
// Bounded waits: a wait that runs out sets the status word and later waits are skipped; the block
// still reaches every block-wide barrier and both cluster barriers. The second cluster barrier
// (arrive right after the deposits, wait before the row ends; in a normal run every peer has
// arrived long before) keeps a block that gave up from exiting while a peer's deposit into its
// shared memory is still to be issued.
//
// SHIFT (one cluster per row, not FULL, not CAUSAL): rows whose byte length is not a multiple of 16,
// in 16-byte aligned tensors. Row i is then covered by the aligned vectors gv0 .. gv0 + nvr - 1 of the
// tensor, starts `head` elements into the first of them and may end inside the last; these two
// vectors are shared with the neighbouring rows. Their foreign elements are replaced by the
// reference identity as they are read (they drop out of the maximum and add 0 to the sum), and
// they are the only vectors stored element by element, own elements only. A bulk copy never
// touches the vector in which the tensor ends: that one is assembled from scalar loads.
template <int DT, bool NEG, bool FULL, bool CAUSAL, bool SHIFT = false>
__global__ void __launch_bounds__(256, 3)
smem_row_kernel(const Params p, const uint32_t stage_bytes, const int slice, const int nchunk_alloc) {
    static_assert(!SHIFT || (!FULL && !CAUSAL), "shifted rows: the general, unmasked variant only");
    constexpr int VE = Traits<DT>::VE;
    constexpr int ESZ = Traits<DT>::ESZ;
    constexpr int U = smem_row_u(DT);
    pdl_launch_dependents();
    extern __shared__ __align__(128) unsigned char smem[];
    __shared__ float2 wp[2][32];
    __shared__ __align__(16) float2 xchg[2][16];
    __shared__ __align__(8) uint64_t xbar[2];
    const int T = blockDim.x, tid = threadIdx.x, lane = tid & 31;
    // A warp owns 32 * U consecutive vectors of a chunk and a lane every 32nd of them: accesses
    // stay coalesced and conflict-free, and the offsets u * US are immediates whatever blockDim is.
    const int tpos = (tid >> 5) * (32 * U) + lane;
    constexpr int US = 32;
    const uint32_t q = cluster_ctarank(), cs = cluster_nctarank();
    const uint32_t ncl = cluster_count_x();
    const uint32_t cid = cluster_id_x();
    const int chunk_vecs = U * T;
    int v0, nv, nchunk;
    int nfill = 0;           // causal: masked vectors of this block's slice, to be filled
    int tail_at = -1;        // causal: local index of the vector that straddles the boundary
    int tail_keep = 0;       //         and how many of its elements are kept
    int64_t gv0 = 0;         // SHIFT: the tensor's vector that holds the row's first element,
    int head = 0;            //        the elements of that vector before the row,
    int nvr = 0;             //        the vectors that cover the row,
    int last_keep = VE;      //        and the elements of the last one up to the row's end
    if (SHIFT) {
        const int64_t e0 = int64_t(cid) * p.cols;
        gv0 = (e0 * ESZ) >> 4;
        head = static_cast<int>(e0 - gv0 * VE);
        nvr = static_cast<int>((head + p.cols + VE - 1) / VE);
        last_keep = static_cast<int>(head + p.cols - int64_t(nvr - 1) * VE);
    }
    if (FULL) {
        v0 = static_cast<int>(q) * slice; nv = slice; nchunk = nchunk_alloc;
    } else {
        const int nvec = SHIFT ? nvr : static_cast<int>(p.nvec);
        v0 = min(nvec, static_cast<int>(q) * slice);
        nv = min(nvec, v0 + slice) - v0;                  // vectors of this block's slice (may be 0)
        if (CAUSAL) {
            const int64_t keep = max(int64_t(0), min(p.cols, int64_t(cid) + p.q_offset + 1));
            const int nvv = static_cast<int>((keep + VE - 1) / VE);        // vectors with a kept element
            const int kept_here = max(0, min(nv, nvv - v0));
            nfill = nv - kept_here;
            nv = kept_here;
            tail_keep = static_cast<int>(keep % VE);
            if (tail_keep != 0 && nv > 0 && v0 + nv == nvv) tail_at = nv - 1;
        }
        nchunk = (nv + chunk_vecs - 1) / chunk_vecs;
    }
    const float ident = ref_identity<NEG>();
    const f32x2 c2 = pair(p.c, p.c);
    uint64_t* bars = reinterpret_cast<uint64_t*>(smem + stage_bytes);
    float* rcs = reinterpret_cast<float*>(smem + stage_bytes + kSmemRowBarBytes) + tid;   // [chunk][thread]
    uint4* sv = reinterpret_cast<uint4*>(smem) + tpos;
    // SHIFT: the row's offset is in gv0 already (one row per cluster) and row_bytes is 0
    const char* xb = static_cast<const char*>(p.x) + (gv0 + v0) * 16;
    uint4* __restrict__ yv = static_cast<uint4*>(p.y) + gv0 + v0 + tpos;
    const int64_t row_bytes = SHIFT ? 0 : p.nvec * 16;

    auto issue_row = [&](int64_t row) {                    // thread 0: one bulk copy per chunk
        for (int ch = 0; ch < nchunk; ++ch) {
            int cv = FULL ? chunk_vecs : min(chunk_vecs, nv - ch * chunk_vecs);
            if (SHIFT && gv0 + v0 + ch * chunk_vecs + cv > p.tensor_vecs) {
                // the tensor ends inside this chunk's last vector: scalar loads for that one, into shared memory
                --cv;
                const int64_t gv = gv0 + v0 + ch * chunk_vecs + cv;
                float t[VE];
#pragma unroll
                for (int i = 0; i < VE; ++i) t[i] = gv * VE + i < p.rows * p.cols ? load_elem<DT>(p.x, gv * VE + i) : 0.0f;
                reinterpret_cast<uint4*>(smem)[ch * chunk_vecs + cv] = pack<DT>(t);
            }
            bulk_load_row(smem_u32(smem) + uint32_t(ch) * uint32_t(chunk_vecs) * 16u,
                          xb + row * row_bytes + int64_t(ch) * chunk_vecs * 16,
                          uint32_t(cv) * 16u, smem_u32(&bars[ch]), p.dbg_extra_tx);
        }
    };

    if (tid == 0) {
        for (int ch = 0; ch < kSmemRowMaxChunks; ++ch) mbar_init(smem_u32(&bars[ch]), 1);
        mbar_init(smem_u32(&xbar[0]), 1);
        mbar_init(smem_u32(&xbar[1]), 1);
        mbar_fence_init();
        fence_proxy_async_smem();
        // (SHIFT: the span may include the vector in which the tensor ends; a prefetch reads nothing)
        pdl_wait_first_wave<true>(cid, p.lag_ns, p.lag_rows, p.early_pf, [&] {
            if (cid < p.rows && nv > 0) pdl_early_prefetch(xb + int64_t(cid) * row_bytes, int64_t(SHIFT ? max(nv - 1, 1) : nv) * 16); });
        if (cid < p.rows) issue_row(cid);
        // the row that starts a fraction of a generation of resident clusters later: its slice is on
        // its way to L2 while this one is worked on
        const int64_t pr = int64_t(cid) + p.pf_rows;
        if (SHIFT) {
            // the later row's own covering vectors, this block's share of them (the last vector left out: see above)
            if (p.pf_rows > 0 && pr < p.rows && nv > 1)
                l2_prefetch(static_cast<const char*>(p.x) + (((pr * p.cols * ESZ) >> 4) + v0) * 16, uint32_t(nv - 1) * 16u);
        } else if (p.pf_rows > 0 && pr < p.rows) {
            int pnv = nv;
            if (CAUSAL) {
                const int64_t pkeep = max(int64_t(0), min(p.cols, pr + p.q_offset + 1));
                const int slice_nv = min(static_cast<int>(p.nvec), v0 + slice) - v0;
                pnv = max(0, min(slice_nv, static_cast<int>((pkeep + VE - 1) / VE) - v0));
            }
            if (pnv > 0) l2_prefetch(xb + pr * row_bytes, uint32_t(pnv) * 16u);
        }
    }
    __syncthreads();
    if (cs > 1) {   // peers are resident, their mbarriers initialised, before any remote deposit
        cluster_arrive_relaxed();
        cluster_wait_acquire();
    }
    pdl_wait();

    if (CAUSAL && nfill > 0 && cid < p.rows) {
        // masked part of this block's slice: +0, written while the kept part is still on its way
        const uint4 zv = make_uint4(0u, 0u, 0u, 0u);
        uint4* yfill = yv - tpos + int64_t(cid) * p.nvec;
        for (int v = nv + tid; v < nv + nfill; v += T) st_stream(yfill + v, zv);
    }

    bool alive = true;      // false once a bounded wait has expired: later waits are skipped
    uint32_t it = 0;
    for (int64_t row = cid; row < p.rows; row += ncl, ++it) {   // the same trip count for the whole cluster
        const int par = static_cast<int>(it & 1u);
        const uint32_t phase = it & 1u;
        if (cs > 1 && tid == 0) mbar_expect_tx(smem_u32(&xbar[par]), cs * 8u);

        // ---- pass 1
        float r = ident, s = 0.0f;
        for (int ch = 0; ch < nchunk; ++ch) {
            // warp 0 polls, the other warps wait at the hardware barrier (no issue slots spent)
            if (tid < 32 && alive) alive = mbar_wait_warp(smem_u32(&bars[ch]), phase, p.status, p.wait_polls);
            if (T > 32) __syncthreads();
            else if (SHIFT) __syncwarp();      // (lane 0 may have written the tensor's last vector itself)
            uint4* sc = sv + ch * chunk_vecs;
            const int cbase = ch * chunk_vecs + tpos;
            if (!FULL) {
                // this thread's vectors of the chunk that lie past the slice's end become identity
                // vectors, so that the arithmetic below needs no bounds (a zero scale, for which
                // 2^(-inf * 0) is NaN, never reaches this variant: the host routes it elsewhere)
                const uint32_t idw = ident_word<DT, NEG>();
#pragma unroll
                for (int u = 0; u < U; ++u)
                    if (cbase + u * US >= nv) sc[u * US] = make_uint4(idw, idw, idw, idw);
            }
            uint4 raw[U];
#pragma unroll
            for (int u = 0; u < U; ++u) raw[u] = sc[u * US];
            if (CAUSAL) {
#pragma unroll
                for (int u = 0; u < U; ++u)
                    if (cbase + u * US == tail_at) mask_tail<DT, NEG>(raw[u], tail_keep);
            }
            // SHIFT: does this chunk hold the row's first or last vector (and is that one shared with a neighbour)?
            // A block-uniform question, so that every other chunk runs the plain code.
            const int vch = v0 + ch * chunk_vecs;
            const bool edge = SHIFT && ((vch == 0 && head > 0) || (last_keep < VE && nvr - 1 >= vch && nvr - 1 < vch + chunk_vecs));
            if (edge) {    // the neighbours' elements drop out
#pragma unroll
                for (int u = 0; u < U; ++u) {
                    const int vr = v0 + cbase + u * US;
                    if (vr == 0 && head > 0) mask_head<DT, NEG>(raw[u], head);
                    if (vr == nvr - 1 && last_keep < VE) mask_tail<DT, NEG>(raw[u], last_keep);
                }
            }
            RefAcc<DT, NEG> ref;
            ref.init();
#pragma unroll
            for (int u = 0; u < U; ++u) ref.fold(raw[u]);
            const float rc = ref.value();
            rcs[ch * T] = rc;
            // all of these elements masked (or none): subtract 0 instead of the identity
            const float ru = (rc == ident) ? 0.0f : rc;
            const f32x2 ru2 = pair(ru, ru);
            f32x2 acc[VE / 2];
#pragma unroll
            for (int k = 0; k < VE / 2; ++k) acc[k] = pair(0.0f, 0.0f);
#pragma unroll
            for (int u = 0; u < U; ++u) sc[u * US] = ex2_vec<DT>(raw[u], ru2, c2, acc);
#pragma unroll
            for (int k = 1; k < VE / 2; ++k) acc[0] = add2(acc[0], acc[k]);
            const float part = pair_sum(acc[0]);
            // online merge of (rc, part) into (r, s): only the reference left behind is rescaled
            const float rn = ref_pick<NEG>(r, rc);
            const bool keep = (rn == r);
            const float lo = keep ? rc : r;
            const float f = (lo == ident) ? 1.0f : ex2_ftz((lo - rn) * p.c);
            s = keep ? fmaf(part, f, s) : fmaf(s, f, part);
            r = rn;
        }
        float R = r;
        block_merge_pairs<NEG>(R, s, wp[par], p.c);
        if (cs > 1) {
            if (tid < cs)
                st_async_v2(map_to_rank(smem_u32(&xchg[par][q]), tid), R, s, map_to_rank(smem_u32(&xbar[par]), tid));
            cluster_arrive_relaxed();          // waited for at the end of the row
            if (tid < 32 && alive) alive = mbar_wait_warp(smem_u32(&xbar[par]), (it >> 1) & 1u, p.status, p.wait_polls);
            if (T > 32) __syncthreads();
            R = ident; s = 0.0f;
            if (lane < static_cast<int>(cs)) ld_shared_v2(smem_u32(&xchg[par][lane]), R, s);
            warp_merge_pairs<NEG>(R, s, p.c);
        }

        // ---- pass 2: scale the stored e, chunk by chunk with the chunk's own reference
        const float inv = recip<DT>(s);
        uint4* yrow = yv + (SHIFT ? int64_t(0) : row * p.nvec);
        for (int ch = 0; ch < nchunk; ++ch) {
            const uint4* sc = sv + ch * chunk_vecs;
            const float rc = rcs[ch * T];
            const float fac = (rc == ident) ? 1.0f : ex2_noflush((rc - R) * p.c);
            // bf16: e carries 2^64 and inv 2^-64; a factor this small is applied separately so
            // that fac * inv cannot underflow before it meets e
            const bool one_mul = DT != DT_BF16 || fac >= 0x1p-40f || !(fac == fac);
            const float f1 = one_mul ? fac * inv : inv;
            const int cbase = ch * chunk_vecs + tpos;
            uint4* yc = yrow + ch * chunk_vecs;
            const f32x2 f2 = pair(f1, f1);
            // SHIFT: the row's first and last vector hold the neighbours' elements too: own elements only, one by one.
            // Only a chunk that holds such a vector takes this path (block-uniform), in a loop that is NOT unrolled:
            // the element-wise stores stay out of the code every other chunk runs (unrolled into it they cost the
            // kernel 15 % more instructions and instruction-fetch stalls: 98 against 80 us on 2048 rows of 50257 bf16 columns).
            const int vch = v0 + ch * chunk_vecs;
            const bool edge = SHIFT && ((vch == 0 && head > 0) || (last_keep < VE && nvr - 1 >= vch && nvr - 1 < vch + chunk_vecs));
            if (edge) {
                const f32x2 g2 = pair(fac, fac);
#pragma unroll 1
                for (int u = 0; u < U; ++u) {
                    if (cbase + u * US >= nv) continue;
                    const uint4 rv = sc[u * US];
                    const uint4 out = (DT == DT_BF16 && !one_mul) ? scale_vec<DT, true>(rv, f2, g2) : scale_vec<DT, false>(rv, f2, f2);
                    const int vr = v0 + cbase + u * US;
                    const int lo = (vr == 0) ? head : 0, hi = (vr == nvr - 1) ? last_keep : VE;
                    if (lo == 0 && hi == VE) {
                        st_stream(yc + u * US, out);
                    } else {
                        float f[VE];
                        unpack<DT>(out, f);
#pragma unroll
                        for (int i = 0; i < VE; ++i)
                            if (i >= lo && i < hi) store_elem<DT>(p.y, (gv0 + vr) * VE + i, f[i]);
                    }
                }
                continue;
            }
            uint4 raw[U];
#pragma unroll
            for (int u = 0; u < U; ++u) raw[u] = sc[u * US];
            if (DT == DT_BF16 && !one_mul) {
                // rare: both multiplications before the one rounding
                const f32x2 g2 = pair(fac, fac);
#pragma unroll
                for (int u = 0; u < U; ++u)
                    if (FULL || cbase + u * US < nv) st_stream(yc + u * US, scale_vec<DT, true>(raw[u], f2, g2));
            } else {
#pragma unroll
                for (int u = 0; u < U; ++u)
                    if (FULL || cbase + u * US < nv) st_stream(yc + u * US, scale_vec<DT, false>(raw[u], f2, f2));
            }
        }

        if (CAUSAL && nfill > 0 && !(0.0f * inv == 0.0f)) {
            // the masked part was filled with +0 up front; a row that turned out NaN (or kept no
            // column: 1/S is infinite) owes it 0 * (1/S) = NaN instead
            float z[VE];
#pragma unroll
            for (int k = 0; k < VE; ++k) z[k] = 0.0f * inv;
            const uint4 zv = pack<DT>(z);
            for (int v = nv + tid; v < nv + nfill; v += T) st_stream(yrow - tpos + v, zv);
        }

        if (cs > 1) cluster_wait_acquire();   // completes at once unless a peer gave up on a wait

        if (!CAUSAL && row + ncl < p.rows) {     // more rows than clusters: the slice is free once everyone has read it
            __syncthreads();
            if (tid == 0) { fence_proxy_async_smem(); issue_row(row + ncl); }
        }
    }
}

// Self-test of the bounded wait: one block arms an mbarrier for 16 bytes that nothing ever copies,
// warp 0 waits for it with the given poll cap, gives up, records DEV_TIMEOUT, and the block still
// meets at its barrier and returns. Nothing is read or written besides the status word.
__global__ void __launch_bounds__(64, 1) wait_probe_kernel(int* status, const int polls) {
    __shared__ __align__(8) uint64_t bar;
    if (threadIdx.x == 0) {
        mbar_init(smem_u32(&bar), 1);
        mbar_fence_init();
        mbar_expect_tx(smem_u32(&bar), 16u);
    }
    __syncthreads();
    if (threadIdx.x < 32) (void)mbar_wait_warp(smem_u32(&bar), 0u, status, polls);
    __syncthreads();
}

}  // namespace fsm
