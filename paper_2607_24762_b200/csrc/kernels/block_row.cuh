// Block-per-row softmax kernels. One pass over the data: every thread keeps
// its share of the row in registers as 2^((x - r_t) c) against its OWN reference r_t (the max of
// its elements), so each element costs one ex2; the (r, s) partial pairs are then merged with the
// online-softmax rule (Milakov-Gimelshein)
//     (r, s) (+) (r', s') = (R = max(r, r'),  s 2^((r-R)c) + s' 2^((r'-R)c))
// across the warp (shuffles) and the block (shared memory, one __syncthreads per row). The output
// is e * 2^((r_t - R)c) / S. (Rows split over a thread-block cluster are in smem_row.cuh, which
// shares block_merge_pairs.)
//
// Two front ends share that arithmetic:
//   block_row_kernel      128-bit global loads straight into registers
//   block_row_tma_kernel  the row brought into shared memory by cp.async.bulk (no multicast),
//                         completion tracked by an mbarrier
#pragma once
#include "common.cuh"

namespace fsm {

// Threads per block the register budget allows for a payload of VPT*VE floats per thread.
template <int DT, int VPT> struct BlockCfg {
    static constexpr int PAYLOAD = VPT * Traits<DT>::VE;
    static constexpr int MAX_THREADS = PAYLOAD <= 16 ? 1024 : 512;
};

// Per-thread part: e[k][i] = 2^((x - r_use) c), r = own reference, s = sum of e.
// valid(k) says whether this thread's k-th vector exists.
template <int DT, bool NEG, int VPT, typename Valid>
__device__ __forceinline__ void thread_partial(const uint4 (&raw)[VPT], float (&e)[VPT][Traits<DT>::VE],
                                               float& r, float& s, float c, Valid valid) {
    constexpr int VE = Traits<DT>::VE;
    RefAcc<DT, NEG> acc;
    acc.init();
#pragma unroll
    for (int k = 0; k < VPT; ++k)
        if (valid(k)) acc.fold(raw[k]);
    r = acc.value();
    // A thread whose elements are all masked (or that has none) subtracts 0 instead of the identity.
    const float r_use = (r == ref_identity<NEG>()) ? 0.0f : r;
    s = 0.0f;
#pragma unroll
    for (int k = 0; k < VPT; ++k) {
        unpack<DT>(raw[k], e[k]);
        if (valid(k)) {
#pragma unroll
            for (int i = 0; i < VE; ++i) {
                e[k][i] = ex2_elem<DT>(e[k][i] - r_use, c);
                s += e[k][i];
            }
        }
    }
}

// Block-wide merge of (r, s). `wp` points at 32 float2 slots; the caller alternates between two
// such arrays from row to row so that one __syncthreads per row is enough.
template <bool NEG>
__device__ __forceinline__ void block_merge_pairs(float& r, float& s, float2* wp, float c) {
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5, nwarps = blockDim.x >> 5;
    warp_merge_pairs<NEG>(r, s, c);
    if (nwarps == 1) return;
    if (lane == 0) wp[warp] = make_float2(r, s);
    __syncthreads();
    const float2 v = (lane < nwarps) ? wp[lane] : make_float2(ref_identity<NEG>(), 0.0f);
    r = v.x; s = v.y;
    warp_merge_pairs<NEG>(r, s, c);
}

template <int DT, bool NEG, int VPT, typename Valid, typename VecIndex>
__device__ __forceinline__ void scale_and_store(float (&e)[VPT][Traits<DT>::VE], float r_t, float R, float S,
                                                float c, uint4* yrow, Valid valid, VecIndex vec) {
    constexpr int VE = Traits<DT>::VE;
    const float fac = ref_factor(r_t, R, c, ref_identity<NEG>());
    const float inv = recip<DT>(S);
    if (DT != DT_BF16 || fac >= 0x1p-40f || !(fac == fac)) {
        const float f = fac * inv;
#pragma unroll
        for (int k = 0; k < VPT; ++k) {
            if (valid(k)) {
#pragma unroll
                for (int i = 0; i < VE; ++i) e[k][i] *= f;
                st_stream(yrow + vec(k), pack<DT>(e[k]));
            }
        }
    } else {
        // bf16 carries a 2^64 bias in e and 2^-64 in inv: with a thread reference far below the
        // row's, fac * inv would underflow although e * inv * fac is a representable (subnormal)
        // bf16 value, so the two factors are applied one after the other.
#pragma unroll
        for (int k = 0; k < VPT; ++k) {
            if (valid(k)) {
#pragma unroll
                for (int i = 0; i < VE; ++i) e[k][i] = (e[k][i] * inv) * fac;
                st_stream(yrow + vec(k), pack<DT>(e[k]));
            }
        }
    }
}

// ---------------------------------------------------------------------------------------------
// block per row, direct global loads
// ---------------------------------------------------------------------------------------------
template <int DT, bool NEG, int VPT>
__global__ void __launch_bounds__(BlockCfg<DT, VPT>::MAX_THREADS, 1)
block_row_kernel(const Params p) {
    constexpr int VE = Traits<DT>::VE;
    __shared__ float2 wp[2][32];
    pdl_launch_dependents();
    const int T = blockDim.x, tid = threadIdx.x;
    const int nvec = static_cast<int>(p.nvec);
    const uint4* __restrict__ xv = static_cast<const uint4*>(p.x);
    uint4* __restrict__ yv = static_cast<uint4*>(p.y);
    auto valid = [&](int k) { return tid + k * T < nvec; };
    auto vec = [&](int k) { return tid + k * T; };
    int par = 0;
    pdl_wait();
    for (int64_t row = blockIdx.x; row < p.rows; row += gridDim.x, par ^= 1) {
        uint4 raw[VPT];
#pragma unroll
        for (int k = 0; k < VPT; ++k) {
            raw[k] = make_uint4(0u, 0u, 0u, 0u);
            if (valid(k)) raw[k] = ld_stream(xv + row * p.nvec + vec(k));
        }
        // one-shot grids: the row of the block that starts half a generation later goes to L2
        if (tid == 0 && p.pf_rows > 0 && row + p.pf_rows < p.rows)
            l2_prefetch(reinterpret_cast<const char*>(xv + (row + p.pf_rows) * p.nvec), uint32_t(nvec) * 16u);
        float e[VPT][VE], r_t, s;
        thread_partial<DT, NEG, VPT>(raw, e, r_t, s, p.c, valid);
        float R = r_t;
        block_merge_pairs<NEG>(R, s, wp[par], p.c);
        scale_and_store<DT, NEG, VPT>(e, r_t, R, s, p.c, yv + row * p.nvec, valid, vec);
    }
}

// ---------------------------------------------------------------------------------------------
// block per row for rows whose byte length is NOT a multiple of 16 (x and y themselves 16-byte
// aligned): the row is read as the aligned 16-byte vectors that cover it. Row i starts `head`
// elements into its first vector and may end inside its last one; those two vectors are shared
// with the neighbouring rows, so their foreign elements are replaced by the reference identity
// (they drop out of the maximum and add 0 to the sum) and they are the only ones stored element by
// element -- a full-vector store there would write the neighbours' outputs. Everything between
// is the block kernel above: 128-bit accesses, one pass, one ex2 per element. The tensor's very
// last vector, when the tensor ends inside it, is assembled from scalar loads: no byte beyond the
// tensor is touched. (A zero scale never comes here: the identity times 0 is NaN.)
// tensor_vecs = whole 16-byte vectors in the tensor.
// ---------------------------------------------------------------------------------------------
template <int DT, bool NEG, int VPT>
__global__ void __launch_bounds__(BlockCfg<DT, VPT>::MAX_THREADS, 1)
block_row_shift_kernel(const Params p, const int64_t tensor_vecs) {
    constexpr int VE = Traits<DT>::VE;
    constexpr int ESZ = Traits<DT>::ESZ;
    __shared__ float2 wp[2][32];
    pdl_launch_dependents();
    const int T = blockDim.x, tid = threadIdx.x;
    const int cols = static_cast<int>(p.cols);
    const uint4* __restrict__ xv = static_cast<const uint4*>(p.x);
    uint4* __restrict__ yv = static_cast<uint4*>(p.y);
    const int64_t total = p.rows * p.cols;
    auto vec = [&](int k) { return tid + k * T; };
    int par = 0;
    pdl_wait();
    for (int64_t row = blockIdx.x; row < p.rows; row += gridDim.x, par ^= 1) {
        const int64_t e0 = row * p.cols;                                  // the row's first element
        const int64_t gv0 = (e0 * ESZ) >> 4;                              // the vector that holds it
        const int head = static_cast<int>(e0 - gv0 * VE);                 // elements of that vector before the row
        const int nvr = (head + cols + VE - 1) / VE;                      // vectors that cover the row
        const int tail_keep = head + cols - (nvr - 1) * VE;               // elements of the last vector up to the row's end
        auto valid = [&](int k) { return tid + k * T < nvr; };
        uint4 raw[VPT];
#pragma unroll
        for (int k = 0; k < VPT; ++k) {
            raw[k] = make_uint4(0u, 0u, 0u, 0u);
            if (valid(k)) {
                const int64_t gv = gv0 + vec(k);
                if (gv < tensor_vecs) {
                    raw[k] = ld_stream(xv + gv);
                } else {                                                  // the tensor ends inside this vector
                    float t[VE];
#pragma unroll
                    for (int i = 0; i < VE; ++i) t[i] = gv * VE + i < total ? load_elem<DT>(p.x, gv * VE + i) : 0.0f;
                    raw[k] = pack<DT>(t);
                }
                if (vec(k) == 0 && head > 0) mask_head<DT, NEG>(raw[k], head);
                if (vec(k) == nvr - 1 && tail_keep < VE) mask_tail<DT, NEG>(raw[k], tail_keep);
            }
        }
        float e[VPT][VE], r_t, s;
        thread_partial<DT, NEG, VPT>(raw, e, r_t, s, p.c, valid);
        float R = r_t;
        block_merge_pairs<NEG>(R, s, wp[par], p.c);
        const float fac = ref_factor(r_t, R, p.c, ref_identity<NEG>());
        const float inv = recip<DT>(s);
        // bf16: e carries 2^64 and inv 2^-64; a factor this small is applied separately (see scale_and_store)
        const bool one_mul = DT != DT_BF16 || fac >= 0x1p-40f || !(fac == fac);
        const float f1 = one_mul ? fac * inv : inv, f2 = one_mul ? 1.0f : fac;
#pragma unroll
        for (int k = 0; k < VPT; ++k) {
            if (valid(k)) {
#pragma unroll
                for (int i = 0; i < VE; ++i) e[k][i] = one_mul ? e[k][i] * f1 : (e[k][i] * f1) * f2;
                const int v = vec(k);
                const int lo = (v == 0) ? head : 0, hi = (v == nvr - 1) ? tail_keep : VE;
                if (lo == 0 && hi == VE) {
                    st_stream(yv + gv0 + v, pack<DT>(e[k]));
                } else {
#pragma unroll
                    for (int i = 0; i < VE; ++i)
                        if (i >= lo && i < hi) store_elem<DT>(p.y, (gv0 + v) * VE + i, e[k][i]);
                }
            }
        }
    }
}

// ---------------------------------------------------------------------------------------------
// Short rows whose byte length is not a multiple of 16 (x and y themselves 16-byte aligned): a
// block takes blockDim.x CONSECUTIVE rows, i.e. one contiguous span of the tensor. The span is read as
// the aligned 16-byte vectors that cover it (coalesced, whole sectors) into shared memory, every
// thread works on its own row there -- the element-wise kernel's arithmetic, thread-local: the
// reference, the sum, then y = 2^((x - R) c) / S written back in place in the element dtype -- and
// the span leaves as 16-byte vectors again. Only the span's first and last vector can be shared
// with the neighbouring blocks: those are stored element by element, own elements only. The
// tensor's very last vector, when the tensor ends inside it, is assembled from scalar loads.
// dynamic shared memory: the span, rounded out to whole vectors. tensor_vecs = whole vectors in the tensor.
// ---------------------------------------------------------------------------------------------
template <int DT> __device__ __forceinline__ float smem_elem(const unsigned char* sm, int i) {
    if constexpr (DT == DT_F32) return reinterpret_cast<const float*>(sm)[i];
    else if constexpr (DT == DT_BF16) return __bfloat162float(reinterpret_cast<const __nv_bfloat16*>(sm)[i]);
    else return __half2float(reinterpret_cast<const __half*>(sm)[i]);
}
template <int DT> __device__ __forceinline__ void smem_put(unsigned char* sm, int i, float v) {
    if constexpr (DT == DT_F32) reinterpret_cast<float*>(sm)[i] = v;
    else if constexpr (DT == DT_BF16) reinterpret_cast<__nv_bfloat16*>(sm)[i] = __float2bfloat16_rn(v);
    else reinterpret_cast<__half*>(sm)[i] = __float2half_rn(v);
}

template <int DT, bool NEG>
__global__ void __launch_bounds__(128)
span_rows_kernel(const Params p, const int64_t tensor_vecs) {
    constexpr int VE = Traits<DT>::VE;
    constexpr int ESZ = Traits<DT>::ESZ;
    extern __shared__ __align__(128) unsigned char smem[];
    pdl_launch_dependents();
    const int T = blockDim.x, tid = threadIdx.x;
    const int cols = static_cast<int>(p.cols);
    const int64_t r0 = int64_t(blockIdx.x) * T;
    const int nr = static_cast<int>(min(int64_t(T), p.rows - r0));          // rows of this block
    const int64_t e0 = r0 * p.cols, e1 = (r0 + nr) * p.cols;                // its elements: [e0, e1)
    const int64_t gv0 = (e0 * ESZ) >> 4, gv1 = (e1 * ESZ + 15) >> 4;        // the vectors that cover them
    const int nv = static_cast<int>(gv1 - gv0);
    const int head = static_cast<int>(e0 - gv0 * VE);                       // elements of the first vector before the span
    const int tail_keep = static_cast<int>(e1 - (gv1 - 1) * VE);            // elements of the last vector inside the span
    const int64_t total = p.rows * p.cols;
    const uint4* __restrict__ xv = static_cast<const uint4*>(p.x);
    uint4* __restrict__ yv = static_cast<uint4*>(p.y);
    uint4* sv = reinterpret_cast<uint4*>(smem);
    pdl_wait();
    for (int vb = tid; vb < nv; vb += 8 * T) {                              // eight loads in flight per thread
        uint4 t8[8];
#pragma unroll
        for (int u = 0; u < 8; ++u) {
            const int v = vb + u * T;
            const int64_t gv = gv0 + v;
            t8[u] = make_uint4(0u, 0u, 0u, 0u);
            if (v < nv && gv < tensor_vecs) t8[u] = ld_stream(xv + gv);
        }
#pragma unroll
        for (int u = 0; u < 8; ++u) {
            const int v = vb + u * T;
            const int64_t gv = gv0 + v;
            if (v < nv) {
                if (gv >= tensor_vecs) {                                    // the tensor ends inside this vector
                    float t[VE];
#pragma unroll
                    for (int i = 0; i < VE; ++i) t[i] = gv * VE + i < total ? load_elem<DT>(p.x, gv * VE + i) : 0.0f;
                    t8[u] = pack<DT>(t);
                }
                sv[v] = t8[u];
            }
        }
    }
    __syncthreads();
    if (tid < nr) {
        const int sb = head + tid * cols;                                   // this thread's row, in elements of the span buffer
        const float ident = ref_identity<NEG>();
        float r = ident;
#pragma unroll 4
        for (int j = 0; j < cols; ++j) r = ref_pick<NEG>(r, smem_elem<DT>(smem, sb + j));
        const float ru = (r == ident) ? 0.0f : r;
        // The sum may flush terms below 2^-126 (the largest term is 1); the outputs may too, except bf16's, whose
        // subnormals are still representable values of the output format.
        float s0 = 0.0f, s1 = 0.0f;                                         // two chains: the additions need not wait for each other
        int j = 0;
#pragma unroll 2
        for (; j + 1 < cols; j += 2) {
            s0 += ex2_ftz((smem_elem<DT>(smem, sb + j) - ru) * p.c);
            s1 += ex2_ftz((smem_elem<DT>(smem, sb + j + 1) - ru) * p.c);
        }
        if (j < cols) s0 += ex2_ftz((smem_elem<DT>(smem, sb + j) - ru) * p.c);
        const float inv = 1.0f / (s0 + s1);
#pragma unroll 4
        for (int j = 0; j < cols; ++j) {
            const float t = (smem_elem<DT>(smem, sb + j) - ru) * p.c;
            smem_put<DT>(smem, sb + j, (DT == DT_BF16 ? ex2_noflush(t) : ex2_ftz(t)) * inv);
        }
    }
    __syncthreads();
    for (int v = tid; v < nv; v += T) {
        const int64_t gv = gv0 + v;
        const int lo = (v == 0) ? head : 0, hi = (v == nv - 1) ? tail_keep : VE;
        if (lo == 0 && hi == VE) {
            st_stream(yv + gv, sv[v]);
        } else {
            for (int i = lo; i < hi; ++i) store_elem<DT>(p.y, gv * VE + i, smem_elem<DT>(smem, v * VE + i));
        }
    }
}

// ---------------------------------------------------------------------------------------------
// block per row, rows staged in a shared-memory ring by bulk async copies
// Every warp waits for the row's mbarrier by itself: one polling warp and a block barrier, the form
// that pays in the split-row kernel, is slower here (fp32 rows of 12 / 16 KiB: 31.6 -> 33.1, 41.0 -> 42.9 us).
// dynamic shared memory: [nstage][stage_bytes] row buffers | nstage mbarriers (8 B each)
// ---------------------------------------------------------------------------------------------
template <int DT, bool NEG, int VPT>
__global__ void __launch_bounds__(BlockCfg<DT, VPT>::MAX_THREADS, 1)
block_row_tma_kernel(const Params p, const int nstage, const uint32_t stage_bytes) {
    constexpr int VE = Traits<DT>::VE;
    pdl_launch_dependents();
    extern __shared__ __align__(128) unsigned char smem[];
    __shared__ float2 wp[2][32];
    const int T = blockDim.x, tid = threadIdx.x;
    const int nvec = static_cast<int>(p.nvec);
    const uint32_t row_bytes = static_cast<uint32_t>(p.nvec) * 16u;
    uint64_t* bars = reinterpret_cast<uint64_t*>(smem + size_t(nstage) * stage_bytes);
    const char* xb = static_cast<const char*>(p.x);
    uint4* __restrict__ yv = static_cast<uint4*>(p.y);
    auto valid = [&](int k) { return tid + k * T < nvec; };
    auto vec = [&](int k) { return tid + k * T; };

    const int64_t first = blockIdx.x;
    const int64_t n_my = first < p.rows ? (p.rows - first + gridDim.x - 1) / gridDim.x : 0;
    if (tid == 0) {
        for (int s = 0; s < nstage; ++s) mbar_init(smem_u32(&bars[s]), 1);
        mbar_fence_init();
        fence_proxy_async_smem();
        pdl_wait_first_wave<false>(first, p.lag_ns, p.lag_rows, p.early_pf, [&] { if (n_my > 0) pdl_early_prefetch(xb + first * row_bytes, row_bytes); });
        for (int s = 0; s < nstage && s < n_my; ++s)
            bulk_load_row(smem_u32(smem + size_t(s) * stage_bytes),
                          xb + (first + int64_t(s) * gridDim.x) * row_bytes, row_bytes, smem_u32(&bars[s]));
    }
    __syncthreads();
    pdl_wait();

    int stage = 0;
    uint32_t phase = 0;
    bool alive = true;      // false once a bounded wait has expired: later waits are skipped
    for (int64_t i = 0; i < n_my; ++i) {
        const int64_t row = first + i * gridDim.x;
        if (alive) alive = mbar_wait_warp(smem_u32(&bars[stage]), phase, p.status);
        const uint4* srow = reinterpret_cast<const uint4*>(smem + size_t(stage) * stage_bytes);
        uint4 raw[VPT];
#pragma unroll
        for (int k = 0; k < VPT; ++k) {
            raw[k] = make_uint4(0u, 0u, 0u, 0u);
            if (valid(k)) raw[k] = srow[vec(k)];
        }
        float e[VPT][VE], r_t, s;
        thread_partial<DT, NEG, VPT>(raw, e, r_t, s, p.c, valid);
        float R = r_t;
        block_merge_pairs<NEG>(R, s, wp[i & 1], p.c);
        // every thread has read its part of this stage (the merge's barrier, or the shuffles of a
        // single-warp block): refill it
        if (tid == 0 && i + nstage < n_my) {
            fence_proxy_async_smem();
            bulk_load_row(smem_u32(smem + size_t(stage) * stage_bytes),
                          xb + (row + int64_t(nstage) * gridDim.x) * row_bytes, row_bytes, smem_u32(&bars[stage]));
        }
        scale_and_store<DT, NEG, VPT>(e, r_t, R, s, p.c, yv + row * p.nvec, valid, vec);
        if (++stage == nstage) { stage = 0; phase ^= 1u; }
    }
}

// ---------------------------------------------------------------------------------------------
// generic: any cols, any alignment, element-wise accesses; reads the row twice (the second read
// normally hits L2). Pass 1 keeps a running (r, s) per thread -- the online update itself.
// ---------------------------------------------------------------------------------------------
template <int DT, bool NEG, bool CAUSAL>
__global__ void __launch_bounds__(1024, 1)
generic_row_kernel(const Params p) {
    __shared__ float2 wp[2][32];
    pdl_launch_dependents();
    pdl_wait();
    const int T = blockDim.x, tid = threadIdx.x;
    const float ident = ref_identity<NEG>();
    int par = 0;
    for (int64_t row = blockIdx.x; row < p.rows; row += gridDim.x, par ^= 1) {
        const int64_t base = row * p.cols;
        // causal: only the first `keep` columns enter; the rest is filled with 0 * (1/S)
        const int64_t keep = CAUSAL ? max(int64_t(0), min(p.cols, row + p.q_offset + 1)) : p.cols;
        float r = ident, s = 0.0f;
        for (int64_t j = tid; j < keep; j += T) {
            const float x = load_elem<DT>(p.x, base + j);
            const float rn = ref_pick<NEG>(r, x);
            const float ru = (rn == ident) ? 0.0f : rn;
            s = s * ref_factor(r, rn, p.c, ident) + ex2_noflush((x - ru) * p.c);
            r = rn;
        }
        block_merge_pairs<NEG>(r, s, wp[par], p.c);
        const float ru = (r == ident) ? 0.0f : r;
        const float inv = 1.0f / s;
        for (int64_t j = tid; j < keep; j += T) {
            const float x = load_elem<DT>(p.x, base + j);
            store_elem<DT>(p.y, base + j, ex2_noflush((x - ru) * p.c) * inv);
        }
        if (CAUSAL) {
            const float fill = 0.0f * inv;
            for (int64_t j = keep + tid; j < p.cols; j += T) store_elem<DT>(p.y, base + j, fill);
        }
    }
}

// ---------------------------------------------------------------------------------------------
// speed-of-light calibration: 16-byte streaming copy, one block per 1024 consecutive vectors
// (four independent loads in flight per thread), blocks handed out by the hardware scheduler
// ---------------------------------------------------------------------------------------------
__global__ void __launch_bounds__(256)
copy_kernel(const uint4* __restrict__ x, uint4* __restrict__ y, const int64_t nvec, const int early_pf) {
    pdl_launch_dependents();
    if (early_pf && threadIdx.x == 0 && int64_t(blockIdx.x) * 1024 < nvec)
        pdl_early_prefetch(reinterpret_cast<const char*>(x + int64_t(blockIdx.x) * 1024), min(int64_t(1024), nvec - int64_t(blockIdx.x) * 1024) * 16);
    pdl_wait();
    for (int64_t base = int64_t(blockIdx.x) * 1024; base < nvec; base += int64_t(gridDim.x) * 1024) {
        uint4 v[4];
#pragma unroll
        for (int u = 0; u < 4; ++u) {
            const int64_t i = base + u * 256 + threadIdx.x;
            if (i < nvec) v[u] = ld_stream(x + i);
        }
#pragma unroll
        for (int u = 0; u < 4; ++u) {
            const int64_t i = base + u * 256 + threadIdx.x;
            if (i < nvec) st_stream(y + i, v[u]);
        }
    }
}

}  // namespace fsm
