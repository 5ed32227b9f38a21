// Shared device helpers for the softmax kernels: 128-bit vector access, dtype unpack/pack,
// base-2 exponential, (reference, sum) pair algebra, warp reductions, mbarrier + bulk-copy PTX.
#pragma once

#include <cuda_bf16.h>
#include <cuda_fp16.h>
#include <cuda_runtime.h>
#include <stdint.h>

namespace fsm {

enum : int { DT_F32 = 0, DT_BF16 = 1, DT_F16 = 2 };

// Status bits a kernel may OR into the per-device status word.
enum : int { DEV_TIMEOUT = 1, DEV_BOUNDS = 2 };
// Poll cap of the bounded waits: about two seconds.
constexpr int kDefaultWaitPolls = 1 << 23;

struct Params {
    const void* x;
    void* y;
    int64_t rows;
    int64_t cols;
    int64_t nvec;      // 16-byte vectors per row (fast kernels: cols * elem_size / 16)
    float c;           // scale * log2(e): exponents are taken in base 2
    int neg;           // c < 0: the row reference is the minimum of x instead of the maximum (host-side dispatch)
    int* status;       // device status word
    int64_t q_offset;  // causal kernels: row i keeps columns j <= i + q_offset
    int64_t pf_rows;   // split-row kernel: the cluster of row i asks L2 for row i + pf_rows (0: off)
    float lag_ns;      // one-shot grids: cluster i < lag_rows starts its loads i * lag_ns late (see first_wave_lag)
    int lag_rows;
    uint32_t dbg_extra_tx;   // 0 in every product call. The wait-expiry self-test arms each chunk barrier of the
                             // split-row kernel for this many bytes more than it copies, so that the waits run out.
    int64_t tensor_vecs;     // kernels on shifted vectors: whole 16-byte vectors in the tensor (the last one may be partial)
    int early_pf;            // first wave: ask L2 for the block's own input before griddepcontrol.wait (see pdl_early_prefetch)
    int wait_polls;          // poll cap of the split-row kernel's bounded waits (kDefaultWaitPolls unless that self-test lowered it)
};

template <int DT> struct Traits;
template <> struct Traits<DT_F32>  { static constexpr int VE = 4; static constexpr int ESZ = 4; };
template <> struct Traits<DT_BF16> { static constexpr int VE = 8; static constexpr int ESZ = 2; };
template <> struct Traits<DT_F16>  { static constexpr int VE = 8; static constexpr int ESZ = 2; };

// ---- checked build ------------------------------------------------------------------------------
// With -DFS_DEBUG_BOUNDS (libfsoftmax_debug.so) every global access of every kernel -- they all go
// through the helpers below -- is checked against the address ranges of the tensors the host
// registered for the launch. An access outside them (or a store into a read-only tensor) is NOT
// performed: it sets DEV_BOUNDS in the table's own flag word, records the first offending address
// and the kernel carries on (a load yields zeros), so an indexing error shows up as a status and an
// address instead of a fault. The stand-in for a memory checker on machines where none can be run.
// The table holds no pointer that device code dereferences: whatever the host uploads (even a stale
// or torn copy, as when two streams launch at once), the worst outcome is a false report.
#ifdef FS_DEBUG_BOUNDS
struct DebugRanges {
    unsigned long long lo[8], hi[8];
    int writable[8];
    int n;                              // 0: nothing registered for this launch, nothing is checked
    int flags;                          // DEV_BOUNDS once an access was refused   } never uploaded: the host
    unsigned long long first_bad;       // 0 until an access was refused           } reads and clears them
};
__device__ DebugRanges g_dbg;
__device__ __forceinline__ bool dbg_ok(const void* p, unsigned long long bytes, bool write) {
    if (g_dbg.n == 0) return true;
    const unsigned long long a = reinterpret_cast<unsigned long long>(p);
    const int n = min(g_dbg.n, 8);
    for (int i = 0; i < n; ++i)
        if (a >= g_dbg.lo[i] && a + bytes <= g_dbg.hi[i] && (!write || g_dbg.writable[i])) return true;
    atomicOr(&g_dbg.flags, DEV_BOUNDS);
    atomicCAS(&g_dbg.first_bad, 0ull, a);
    return false;
}
#define FS_DBG_LOAD(p, bytes, zero)  do { if (!dbg_ok((p), (bytes), false)) return zero; } while (0)
#define FS_DBG_STORE(p, bytes)       do { if (!dbg_ok((p), (bytes), true)) return; } while (0)
#define FS_DBG_TOUCH(p)              do { if (!dbg_ok((p), 0, false)) return; } while (0)
#else
#define FS_DBG_LOAD(p, bytes, zero)  do { } while (0)
#define FS_DBG_STORE(p, bytes)       do { } while (0)
#define FS_DBG_TOUCH(p)              do { } while (0)
#endif

// ---- 128-bit streaming global access (every byte is touched once: evict-first) -------------

__device__ __forceinline__ uint4 ld_stream(const uint4* p) {
    FS_DBG_LOAD(p, 16, make_uint4(0u, 0u, 0u, 0u));
    uint4 v;
    asm volatile("ld.global.cs.v4.u32 {%0,%1,%2,%3}, [%4];"
                 : "=r"(v.x), "=r"(v.y), "=r"(v.z), "=r"(v.w) : "l"(p));
    return v;
}

__device__ __forceinline__ void st_stream(uint4* p, const uint4& v) {
    FS_DBG_STORE(p, 16);
    asm volatile("st.global.cs.v4.u32 [%0], {%1,%2,%3,%4};"
                 :: "l"(p), "r"(v.x), "r"(v.y), "r"(v.z), "r"(v.w) : "memory");
}

// 32 bytes at a 32-byte-aligned address in one instruction (256-bit global stores: sm_100): a warp
// whose lanes each own 32 consecutive output bytes writes 1 KiB of whole sectors per instruction,
// where two 16-byte stores per lane each fill half of every sector they touch.
__device__ __forceinline__ void st_stream32(uint4* p, const uint4& a, const uint4& b) {
    FS_DBG_STORE(p, 32);
    asm volatile("st.global.cs.v8.b32 [%0], {%1,%2,%3,%4,%5,%6,%7,%8};"
                 :: "l"(p), "r"(a.x), "r"(a.y), "r"(a.z), "r"(a.w), "r"(b.x), "r"(b.y), "r"(b.z), "r"(b.w) : "memory");
}

__device__ __forceinline__ uint4 ld_shared_v4(uint32_t addr) {
    uint4 v;
    asm volatile("ld.shared.v4.u32 {%0,%1,%2,%3}, [%4];"
                 : "=r"(v.x), "=r"(v.y), "=r"(v.z), "=r"(v.w) : "r"(addr));
    return v;
}

// One 32-bit word of reference identities (one fp32, or two 16-bit elements).
template <int DT, bool NEG>
__device__ __forceinline__ uint32_t ident_word() {
    if constexpr (DT == DT_F32) return NEG ? 0x7f800000u : 0xff800000u;
    else if constexpr (DT == DT_BF16) return NEG ? 0x7f807f80u : 0xff80ff80u;
    else return NEG ? 0x7c007c00u : 0xfc00fc00u;
}

// Causal tail: keep the first `keep` elements (1 .. VE-1) of a vector, set the rest to the
// reference identity (-inf, or +inf when the reference is a minimum) so that they drop out.
template <int DT, bool NEG>
__device__ __forceinline__ void mask_tail(uint4& v, int keep) {
    uint32_t* w = reinterpret_cast<uint32_t*>(&v);
    if constexpr (DT == DT_F32) {
        const uint32_t id = NEG ? 0x7f800000u : 0xff800000u;
#pragma unroll
        for (int k = 0; k < 4; ++k) if (k >= keep) w[k] = id;
    } else {
        const uint32_t id16 = (DT == DT_BF16) ? (NEG ? 0x7f80u : 0xff80u) : (NEG ? 0x7c00u : 0xfc00u);
#pragma unroll
        for (int k = 0; k < 4; ++k) {
            if (2 * k >= keep) w[k] = id16 | (id16 << 16);
            else if (2 * k + 1 >= keep) w[k] = (w[k] & 0xffffu) | (id16 << 16);
        }
    }
}

// The mirror image: the first `skip` elements (1 .. VE-1) become the reference identity.
template <int DT, bool NEG>
__device__ __forceinline__ void mask_head(uint4& v, int skip) {
    uint32_t* w = reinterpret_cast<uint32_t*>(&v);
    if constexpr (DT == DT_F32) {
        const uint32_t id = NEG ? 0x7f800000u : 0xff800000u;
#pragma unroll
        for (int k = 0; k < 4; ++k) if (k < skip) w[k] = id;
    } else {
        const uint32_t id16 = (DT == DT_BF16) ? (NEG ? 0x7f80u : 0xff80u) : (NEG ? 0x7c00u : 0xfc00u);
#pragma unroll
        for (int k = 0; k < 4; ++k) {
            if (2 * k + 1 < skip) w[k] = id16 | (id16 << 16);
            else if (2 * k < skip) w[k] = (w[k] & 0xffff0000u) | id16;
        }
    }
}

// ---- dtype unpack / pack of one 16-byte vector ------------------------------------------------

template <int DT>
__device__ __forceinline__ void unpack(const uint4& v, float (&f)[Traits<DT>::VE]) {
    if constexpr (DT == DT_F32) {
        f[0] = __uint_as_float(v.x); f[1] = __uint_as_float(v.y);
        f[2] = __uint_as_float(v.z); f[3] = __uint_as_float(v.w);
    } else if constexpr (DT == DT_BF16) {
        // bfloat16 is the high half of a binary32 pattern
        f[0] = __uint_as_float(v.x << 16); f[1] = __uint_as_float(v.x & 0xffff0000u);
        f[2] = __uint_as_float(v.y << 16); f[3] = __uint_as_float(v.y & 0xffff0000u);
        f[4] = __uint_as_float(v.z << 16); f[5] = __uint_as_float(v.z & 0xffff0000u);
        f[6] = __uint_as_float(v.w << 16); f[7] = __uint_as_float(v.w & 0xffff0000u);
    } else {
        const __half2* h = reinterpret_cast<const __half2*>(&v);
#pragma unroll
        for (int i = 0; i < 4; ++i) {
            const float2 t = __half22float2(h[i]);
            f[2 * i] = t.x; f[2 * i + 1] = t.y;
        }
    }
}

// Round-to-nearest-even to the stored dtype.
template <int DT>
__device__ __forceinline__ uint4 pack(const float (&f)[Traits<DT>::VE]) {
    uint4 v;
    if constexpr (DT == DT_F32) {
        v.x = __float_as_uint(f[0]); v.y = __float_as_uint(f[1]);
        v.z = __float_as_uint(f[2]); v.w = __float_as_uint(f[3]);
    } else if constexpr (DT == DT_BF16) {
        __nv_bfloat162 a = __floats2bfloat162_rn(f[0], f[1]);
        __nv_bfloat162 b = __floats2bfloat162_rn(f[2], f[3]);
        __nv_bfloat162 c = __floats2bfloat162_rn(f[4], f[5]);
        __nv_bfloat162 d = __floats2bfloat162_rn(f[6], f[7]);
        v.x = *reinterpret_cast<uint32_t*>(&a); v.y = *reinterpret_cast<uint32_t*>(&b);
        v.z = *reinterpret_cast<uint32_t*>(&c); v.w = *reinterpret_cast<uint32_t*>(&d);
    } else {
        __half2 a = __floats2half2_rn(f[0], f[1]);
        __half2 b = __floats2half2_rn(f[2], f[3]);
        __half2 c = __floats2half2_rn(f[4], f[5]);
        __half2 d = __floats2half2_rn(f[6], f[7]);
        v.x = *reinterpret_cast<uint32_t*>(&a); v.y = *reinterpret_cast<uint32_t*>(&b);
        v.z = *reinterpret_cast<uint32_t*>(&c); v.w = *reinterpret_cast<uint32_t*>(&d);
    }
    return v;
}

template <int DT> __device__ __forceinline__ float load_elem(const void* p, int64_t i) {
    FS_DBG_LOAD(static_cast<const char*>(p) + i * Traits<DT>::ESZ, Traits<DT>::ESZ, 0.0f);
    if constexpr (DT == DT_F32) return static_cast<const float*>(p)[i];
    else if constexpr (DT == DT_BF16) return __bfloat162float(static_cast<const __nv_bfloat16*>(p)[i]);
    else return __half2float(static_cast<const __half*>(p)[i]);
}

template <int DT> __device__ __forceinline__ void store_elem(void* p, int64_t i, float v) {
    FS_DBG_STORE(static_cast<char*>(p) + i * Traits<DT>::ESZ, Traits<DT>::ESZ);
    if constexpr (DT == DT_F32) static_cast<float*>(p)[i] = v;
    else if constexpr (DT == DT_BF16) static_cast<__nv_bfloat16*>(p)[i] = __float2bfloat16_rn(v);
    else static_cast<__half*>(p)[i] = __float2half_rn(v);
}

// ---- packed pairs of binary32 -----------------------------------------------------------------
// sm_100 has two-wide fp32 arithmetic on 64-bit register pairs (add/sub/mul/fma .f32x2): the same
// IEEE results as the scalar forms, one issue slot for two elements. These kernels are bound by
// instruction issue long before the fp32 pipe is full, so everything per element that is not the
// exponential itself goes through the pairs.

typedef uint64_t f32x2;

__device__ __forceinline__ f32x2 pair(float lo, float hi) {
    f32x2 r;
    asm("mov.b64 %0, {%1, %2};" : "=l"(r) : "f"(lo), "f"(hi));
    return r;
}
__device__ __forceinline__ f32x2 pair_bits(uint32_t lo, uint32_t hi) {
    f32x2 r;
    asm("mov.b64 %0, {%1, %2};" : "=l"(r) : "r"(lo), "r"(hi));
    return r;
}
__device__ __forceinline__ void unpair(f32x2 v, float& lo, float& hi) {
    asm("mov.b64 {%0, %1}, %2;" : "=f"(lo), "=f"(hi) : "l"(v));
}
__device__ __forceinline__ void unpair_bits(f32x2 v, uint32_t& lo, uint32_t& hi) {
    asm("mov.b64 {%0, %1}, %2;" : "=r"(lo), "=r"(hi) : "l"(v));
}
__device__ __forceinline__ f32x2 add2(f32x2 a, f32x2 b) {
    f32x2 r;
    asm("add.rn.f32x2 %0, %1, %2;" : "=l"(r) : "l"(a), "l"(b));
    return r;
}
__device__ __forceinline__ f32x2 sub2(f32x2 a, f32x2 b) {
    f32x2 r;
    asm("sub.rn.f32x2 %0, %1, %2;" : "=l"(r) : "l"(a), "l"(b));
    return r;
}
__device__ __forceinline__ f32x2 mul2(f32x2 a, f32x2 b) {
    f32x2 r;
    asm("mul.rn.f32x2 %0, %1, %2;" : "=l"(r) : "l"(a), "l"(b));
    return r;
}
__device__ __forceinline__ f32x2 fma2(f32x2 a, f32x2 b, f32x2 c) {
    f32x2 r;
    asm("fma.rn.f32x2 %0, %1, %2, %3;" : "=l"(r) : "l"(a), "l"(b), "l"(c));
    return r;
}
__device__ __forceinline__ float pair_sum(f32x2 v) {
    float lo, hi;
    unpair(v, lo, hi);
    return lo + hi;
}

// Two binary32 values to one word of two bf16 / fp16 (round to nearest even), low element first.
__device__ __forceinline__ uint32_t pack_bf16x2(float lo, float hi) {
    uint32_t r;
    asm("cvt.rn.bf16x2.f32 %0, %1, %2;" : "=r"(r) : "f"(hi), "f"(lo));
    return r;
}
__device__ __forceinline__ uint32_t pack_f16x2(float lo, float hi) {
    uint32_t r;
    asm("cvt.rn.f16x2.f32 %0, %1, %2;" : "=r"(r) : "f"(hi), "f"(lo));
    return r;
}

// One word of two 16-bit elements to a pair of binary32.
template <int DT>
__device__ __forceinline__ f32x2 widen_word(uint32_t w) {
    if constexpr (DT == DT_BF16) {
        return pair_bits(w << 16, w & 0xffff0000u);
    } else {
        const float2 t = __half22float2(*reinterpret_cast<const __half2*>(&w));
        return pair(t.x, t.y);
    }
}

// ---- base-2 exponential on the special-function unit ---------------------------------------
// e = 2^t with t = (x - r) * c <= 0 for the row (or thread) reference r. One MUFU.EX2 per element:
// the flushing form of ex2.approx is a single instruction, the non-flushing one costs three more.
//
// bfloat16 shares binary32's exponent range, so an output below 2^-126 is still a representable
// (subnormal) bf16 value and must not be flushed. bf16 therefore evaluates 2^(t + 64): nothing
// above 2^-190 is flushed, the common factor 2^64 is carried by the row sum and cancels in the
// final e * (1/S) product, which is an ordinary (non-flushing) multiply. The bias costs nothing
// (it is the addend of the fused multiply-add) but rounds t to the spacing of numbers near 64
// (relative error ~3e-6 on e): harmless at 8 bits of output precision, not at fp32's 1e-6
// absolute bound, so fp32 and fp16 (whose subnormals are normal binary32 numbers) use t as is.
template <int DT>
__device__ __forceinline__ float ex2_elem(float d, float c) {
    float t, r;
    if constexpr (DT == DT_BF16) t = fmaf(d, c, 64.0f);
    else                         t = d * c;
    asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(r) : "f"(t));
    return r;
}

__device__ __forceinline__ float ex2_ftz(float t) {
    float r;
    asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(r) : "f"(t));
    return r;
}

// The same for a pair: d = x - r and t = d c (+ 64 for bf16) are two-wide, the exponentials are not.
template <int DT>
__device__ __forceinline__ f32x2 ex2_pair(f32x2 x, f32x2 r2, f32x2 c2) {
    const f32x2 d = sub2(x, r2);
    f32x2 t;
    if constexpr (DT == DT_BF16) t = fma2(d, c2, pair(64.0f, 64.0f));
    else                         t = mul2(d, c2);
    float lo, hi;
    unpair(t, lo, hi);
    return pair(ex2_ftz(lo), ex2_ftz(hi));
}

// e = 2^((x - r) c) for one 16-byte vector of x: each pair of e is added to its own accumulator
// (unrounded), and e comes back in the element dtype, rounded to nearest even.
template <int DT>
__device__ __forceinline__ uint4 ex2_vec(const uint4& raw, f32x2 r2, f32x2 c2, f32x2 (&acc)[Traits<DT>::VE / 2]) {
    const uint32_t w[4] = {raw.x, raw.y, raw.z, raw.w};
    uint32_t o[4];
    if constexpr (DT == DT_F32) {
#pragma unroll
        for (int k = 0; k < 2; ++k) {
            const f32x2 e = ex2_pair<DT>(pair_bits(w[2 * k], w[2 * k + 1]), r2, c2);
            acc[k] = add2(acc[k], e);
            unpair_bits(e, o[2 * k], o[2 * k + 1]);
        }
    } else {
#pragma unroll
        for (int k = 0; k < 4; ++k) {
            const f32x2 e = ex2_pair<DT>(widen_word<DT>(w[k]), r2, c2);
            acc[k] = add2(acc[k], e);
            float lo, hi;
            unpair(e, lo, hi);
            o[k] = DT == DT_BF16 ? pack_bf16x2(lo, hi) : pack_f16x2(lo, hi);
        }
    }
    return make_uint4(o[0], o[1], o[2], o[3]);
}

// y = e * f (TWO: e * f * g, rounded once) for one 16-byte vector of stored e (element dtype),
// rounded to nearest even.
template <int DT, bool TWO>
__device__ __forceinline__ uint4 scale_vec(const uint4& raw, f32x2 f2, f32x2 g2) {
    const uint32_t w[4] = {raw.x, raw.y, raw.z, raw.w};
    uint32_t o[4];
    if constexpr (DT == DT_F32) {
#pragma unroll
        for (int k = 0; k < 2; ++k) {
            f32x2 v = mul2(pair_bits(w[2 * k], w[2 * k + 1]), f2);
            if (TWO) v = mul2(v, g2);
            unpair_bits(v, o[2 * k], o[2 * k + 1]);
        }
    } else {
#pragma unroll
        for (int k = 0; k < 4; ++k) {
            f32x2 v = mul2(widen_word<DT>(w[k]), f2);
            if (TWO) v = mul2(v, g2);
            float lo, hi;
            unpair(v, lo, hi);
            o[k] = DT == DT_BF16 ? pack_bf16x2(lo, hi) : pack_f16x2(lo, hi);
        }
    }
    return make_uint4(o[0], o[1], o[2], o[3]);
}

__device__ __forceinline__ float ex2_noflush(float t) {
    float r;
    asm("ex2.approx.f32 %0, %1;" : "=f"(r) : "f"(t));
    return r;
}

// 1/S. fp32 output: IEEE division. 16-bit output: the special-function unit's reciprocal
// (1 ulp of binary32, far below half an ulp of the output format).
template <int DT>
__device__ __forceinline__ float recip(float s) {
    if constexpr (DT == DT_F32) return 1.0f / s;
    float r;
    asm("rcp.approx.ftz.f32 %0, %1;" : "=f"(r) : "f"(s));
    return r;
}

// ---- row reference (max of x, or min when the scale is negative) ----------------------------

template <bool NEG> __device__ __forceinline__ float ref_identity() {
    return NEG ? __int_as_float(0x7f800000) : __int_as_float(0xff800000);
}
template <bool NEG> __device__ __forceinline__ float ref_pick(float a, float b) {
    return NEG ? fminf(a, b) : fmaxf(a, b);
}

// Running reference over raw 16-byte vectors. fp32 folds element by element; the 16-bit types
// fold two elements per instruction with the packed min/max (exact: the max of two bf16/fp16
// values is one of them; a NaN operand is dropped, as fmaxf does).
template <int DT, bool NEG> struct RefAcc;

template <bool NEG> struct RefAcc<DT_F32, NEG> {
    float a;
    __device__ __forceinline__ void init() { a = ref_identity<NEG>(); }
    __device__ __forceinline__ void fold(const uint4& v) {
        a = ref_pick<NEG>(a, __uint_as_float(v.x)); a = ref_pick<NEG>(a, __uint_as_float(v.y));
        a = ref_pick<NEG>(a, __uint_as_float(v.z)); a = ref_pick<NEG>(a, __uint_as_float(v.w));
    }
    __device__ __forceinline__ float value() const { return a; }
};

template <bool NEG> struct RefAcc<DT_BF16, NEG> {
    uint32_t a;
    static __device__ __forceinline__ uint32_t pk(uint32_t x, uint32_t y) {
        uint32_t r;
        if constexpr (NEG) asm("min.bf16x2 %0, %1, %2;" : "=r"(r) : "r"(x), "r"(y));
        else               asm("max.bf16x2 %0, %1, %2;" : "=r"(r) : "r"(x), "r"(y));
        return r;
    }
    __device__ __forceinline__ void init() { a = NEG ? 0x7f807f80u : 0xff80ff80u; }
    __device__ __forceinline__ void fold(const uint4& v) { a = pk(pk(a, v.x), pk(pk(v.y, v.z), v.w)); }
    __device__ __forceinline__ float value() const {
        return ref_pick<NEG>(__uint_as_float(a << 16), __uint_as_float(a & 0xffff0000u));
    }
};

template <bool NEG> struct RefAcc<DT_F16, NEG> {
    uint32_t a;
    static __device__ __forceinline__ uint32_t pk(uint32_t x, uint32_t y) {
        uint32_t r;
        if constexpr (NEG) asm("min.f16x2 %0, %1, %2;" : "=r"(r) : "r"(x), "r"(y));
        else               asm("max.f16x2 %0, %1, %2;" : "=r"(r) : "r"(x), "r"(y));
        return r;
    }
    __device__ __forceinline__ void init() { a = NEG ? 0x7c007c00u : 0xfc00fc00u; }
    __device__ __forceinline__ void fold(const uint4& v) { a = pk(pk(a, v.x), pk(pk(v.y, v.z), v.w)); }
    __device__ __forceinline__ float value() const {
        const float2 t = __half22float2(*reinterpret_cast<const __half2*>(&a));
        return ref_pick<NEG>(t.x, t.y);
    }
};

// Factor that moves a partial sum taken against reference `r` to the reference `R`
// (R = pick(r, ...)). A partial whose reference is still the identity has sum 0 (or NaN) and keeps
// it: returning 1 avoids inf - inf and 0 * inf for rows that are partly or wholly masked.
__device__ __forceinline__ float ref_factor(float r, float R, float c, float ident) {
    return (r == R || r == ident) ? 1.0f : ex2_noflush((r - R) * c);
}

template <int WIDTH, bool NEG>
__device__ __forceinline__ float warp_pick(float v) {
#pragma unroll
    for (int o = WIDTH / 2; o > 0; o >>= 1) v = ref_pick<NEG>(v, __shfl_xor_sync(0xffffffffu, v, o));
    return v;
}

template <int WIDTH>
__device__ __forceinline__ float warp_sum(float v) {
#pragma unroll
    for (int o = WIDTH / 2; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
    return v;
}

// Merge (r, s) pairs across the 32 lanes of a warp:
//   R = pick_l r_l,  S = sum_l s_l * 2^((r_l - R) c)      (online-softmax merge, Milakov-Gimelshein)
template <bool NEG>
__device__ __forceinline__ void warp_merge_pairs(float& r, float& s, float c) {
    const float R = warp_pick<32, NEG>(r);
    s = warp_sum<32>(s * ref_factor(r, R, c, ref_identity<NEG>()));
    r = R;
}

// ---- shared-memory addresses, mbarrier, bulk async copy (non-multicast) ---------------------

__device__ __forceinline__ uint32_t smem_u32(const void* p) {
    return static_cast<uint32_t>(__cvta_generic_to_shared(p));
}

__device__ __forceinline__ void mbar_init(uint32_t bar, uint32_t count) {
    asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" :: "r"(bar), "r"(count) : "memory");
}

__device__ __forceinline__ void mbar_fence_init() {
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
}

__device__ __forceinline__ void fence_proxy_async_smem() {
    asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
}

__device__ __forceinline__ void mbar_expect_tx(uint32_t bar, uint32_t bytes) {
    asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" :: "r"(bar), "r"(bytes) : "memory");
}

// Global -> this block's shared memory, completion counted in bytes on `bar`.
// dst, src and bytes must be multiples of 16.
__device__ __forceinline__ void bulk_load(uint32_t dst, const void* src, uint32_t bytes, uint32_t bar) {
#ifdef FS_DEBUG_BOUNDS
    if (!dbg_ok(src, bytes, false)) {       // refused: complete the barrier's byte count without copying
        asm volatile("mbarrier.complete_tx.shared::cta.b64 [%0], %1;" :: "r"(bar), "r"(bytes) : "memory");
        return;
    }
#endif
    asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];"
                 :: "r"(dst), "l"(src), "r"(bytes), "r"(bar) : "memory");
}

// Arms `bar` for `bytes` and issues the copy in pieces of at most 32 KiB. The expected byte count
// and the copied byte count come from the same loop (`extra` is zero except in the wait-expiry self-test).
__device__ __forceinline__ void bulk_load_row(uint32_t dst, const char* src, uint32_t bytes, uint32_t bar, uint32_t extra = 0u) {
    mbar_expect_tx(bar, bytes + extra);
    for (uint32_t off = 0; off < bytes; off += 32768u) {
        const uint32_t n = min(32768u, bytes - off);
        bulk_load(dst + off, src + off, n, bar);
    }
}

// Asks the L2 cache for `bytes` (a multiple of 16) at `src`: no destination, nothing to wait for.
__device__ __forceinline__ void l2_prefetch(const char* src, uint32_t bytes) {
    FS_DBG_TOUCH(src);                      // a prefetch must at least start inside a registered tensor
    for (uint32_t off = 0; off < bytes; off += 32768u) {
        const uint32_t n = min(32768u, bytes - off);
        asm volatile("cp.async.bulk.prefetch.L2.global [%0], %1;" :: "l"(src + off), "r"(n) : "memory");
    }
}

// ---- programmatic dependent launch ------------------------------------------------------------
// Every kernel lets the next kernel in the stream be scheduled as soon as all of its own blocks
// have started (launch_dependents), and touches global memory only after the previous kernel has
// completed and flushed (wait). With the launch attribute set by the host this overlaps the next
// launch's latency and prologue with this kernel's tail; without it both are no-ops.

__device__ __forceinline__ void pdl_launch_dependents() { asm volatile("griddepcontrol.launch_dependents;" ::: "memory"); }
__device__ __forceinline__ void pdl_wait() { asm volatile("griddepcontrol.wait;" ::: "memory"); }

// What a block may do before griddepcontrol.wait. Under programmatic dependent launch the blocks of
// a grid become resident while the previous kernel of the stream drains, and wait there until that
// kernel has completed, because it may be the producer of x. Reading x is therefore not allowed
// yet -- but asking L2 for it is: a prefetch has no architectural effect, and L2 is the point of
// coherence, so whatever the previous kernel still writes to those lines lands in the prefetched
// copy. When x is not being rewritten (a train of independent calls) the first wave's loads then
// hit L2 instead of starting DRAM reads only after the previous grid's last store. Measured on B200,
// 256 rows of 512 KiB bf16 in a train of launches: 47.7 -> 46.4 us.
__device__ __forceinline__ void pdl_early_prefetch(const char* src, int64_t bytes) {
    l2_prefetch(src, static_cast<uint32_t>(min(bytes, int64_t(1) << 20)));
}

// The first wave of a one-shot grid starts everywhere at once: every resident cluster loads, then
// every one computes (DRAM idle), then every one stores, and only later generations drift apart
// and overlap. Cluster i of that first wave therefore starts its loads i * lag_ns late, lag_ns
// being the time DRAM needs for one cluster's input: the requests reach DRAM in the order it could
// serve them anyway (the earlier clusters' rows keep it busy), and the wave comes out of its load
// phase already spread over one load time. Later clusters (i >= lag_rows) start as slots free up.
__device__ __forceinline__ void first_wave_lag(int64_t cluster, float lag_ns, int lag_rows) {
    if (lag_ns > 0.0f && cluster > 0 && cluster < lag_rows) __nanosleep(static_cast<uint32_t>(float(cluster) * lag_ns));
}

// Thread 0 of a first-wave cluster (or block) of a one-shot grid, before its first load. With the early
// prefetch on, the lag comes first (the prefetches reach DRAM paced like the loads would, so an
// isolated launch, whose blocks all start at once, loses nothing), then the prefetch and the
// dependency wait. HALF_LAG_AFTER (the split-row kernels): half the lag again after the wait keeps
// the wave's compute phases apart. Measured on B200 in trains of launches, 256 rows of 512 KiB bf16
// through the split-row kernel: 47.6 us without the prefetch; 46.2 with prefetch, wait, whole lag
// (which costs an isolated launch 2 us); 46.5 with lag, prefetch, wait; 45.85 with the half lag added.
// fp32 rows of 16 / 32 KiB through the block kernel fed by bulk copies: 41.9 -> 41.0 and 44.1 -> 43.3 us.
// The four-rows-per-block kernels keep their plain wait-then-lag: there the paced prefetch loses
// (bf16 rows of 10 / 12.5 KiB: 52.8 -> 53.5 and 34.7 -> 37.0 us) and the unpaced one, 1.5-3 % faster in
// a train, costs an isolated launch 1-3 us.
template <bool HALF_LAG_AFTER, class F>
__device__ __forceinline__ void pdl_wait_first_wave(int64_t unit, float lag_ns, int lag_rows, int early_pf, F prefetch) {
    if (early_pf) {
        first_wave_lag(unit, lag_ns, lag_rows);
        if (unit < lag_rows) prefetch();
    }
    pdl_wait();
    if (!early_pf || HALF_LAG_AFTER) first_wave_lag(unit, early_pf ? 0.5f * lag_ns : lag_ns, lag_rows);
}

// Bounded wait on an mbarrier phase. A failed try_wait comes back after a short hardware-defined
// time whatever hint it is given, and a lane that polls back to back burns issue slots the other
// blocks on the SM need (measured: hundreds of instructions per wait). So the first polls are
// immediate (later chunks of a row have usually landed) and the following ones are spaced by
// nanosleep, doubling up to 256 ns. At most `cap` polls (2^23, about two seconds, unless a self-test
// passes less). Measured on 256 rows of 512 KiB bf16 (47.1 us): spacings from none at all to
// 32..128 ns change the time by less than 1%, 128..512 ns costs 4% and 256..1024 ns 9% (every row
// has three waits on its critical path). The cap is an argument, never a memory word: a version of this loop that looked at a
// cap in global memory, even only on every 64th poll, made the split-row kernel 7% slower (256 rows
// of 512 KiB: 50.4 us against 47.1). Returns false (and records DEV_TIMEOUT) if the phase did not
// complete; the caller carries on, skipping further waits, so that every block-wide and
// cluster-wide barrier is still reached and the kernel ends.
__device__ __forceinline__ bool mbar_try(uint32_t bar, uint32_t parity) {
    uint32_t done;
    asm volatile("{\n\t.reg .pred p;\n\t"
                 "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\t"
                 "selp.u32 %0, 1, 0, p;\n\t}"
                 : "=r"(done) : "r"(bar), "r"(parity) : "memory");
    return done != 0;
}

__device__ __forceinline__ bool mbar_wait(uint32_t bar, uint32_t parity, int* status, int cap = kDefaultWaitPolls) {
    if (mbar_try(bar, parity)) return true;
    unsigned ns = 32;
    for (int it = 0; it < cap; ++it) {
        __nanosleep(ns);
        if (mbar_try(bar, parity)) return true;
        if (ns < 256) ns <<= 1;
    }
    atomicOr(status, DEV_TIMEOUT);
    return false;
}

// One lane per warp polls (spinning threads cost issue slots that other blocks' warps need); the
// result is broadcast so that the whole warp agrees on whether the wait expired.
__device__ __forceinline__ bool mbar_wait_warp(uint32_t bar, uint32_t parity, int* status, int cap = kDefaultWaitPolls) {
    int ok = 1;
    if ((threadIdx.x & 31) == 0) ok = mbar_wait(bar, parity, status, cap) ? 1 : 0;
    return __shfl_sync(0xffffffffu, ok, 0) != 0;
}

// ---- thread-block cluster ------------------------------------------------------------------

__device__ __forceinline__ uint32_t cluster_ctarank() {
    uint32_t r; asm volatile("mov.u32 %0, %%cluster_ctarank;" : "=r"(r)); return r;
}
__device__ __forceinline__ uint32_t cluster_nctarank() {
    uint32_t r; asm volatile("mov.u32 %0, %%cluster_nctarank;" : "=r"(r)); return r;
}
__device__ __forceinline__ uint32_t cluster_id_x() {
    uint32_t r; asm volatile("mov.u32 %0, %%clusterid.x;" : "=r"(r)); return r;
}
__device__ __forceinline__ uint32_t cluster_count_x() {
    uint32_t r; asm volatile("mov.u32 %0, %%nclusterid.x;" : "=r"(r)); return r;
}
// Address of `local_addr` (a shared::cta address of this block) in block `rank` of the cluster.
__device__ __forceinline__ uint32_t map_to_rank(uint32_t local_addr, uint32_t rank) {
    uint32_t a; asm volatile("mapa.shared::cluster.u32 %0, %1, %2;" : "=r"(a) : "r"(local_addr), "r"(rank)); return a;
}
// Asynchronous store of two floats into a peer block's shared memory; the 8 bytes are counted as
// a transaction on the peer's mbarrier `mbar` (both addresses are shared::cluster addresses).
__device__ __forceinline__ void st_async_v2(uint32_t addr, float a, float b, uint32_t mbar) {
    asm volatile("st.async.weak.shared::cluster.mbarrier::complete_tx::bytes.v2.f32 [%0], {%1, %2}, [%3];"
                 :: "r"(addr), "f"(a), "f"(b), "r"(mbar) : "memory");
}
__device__ __forceinline__ void ld_shared_v2(uint32_t addr, float& a, float& b) {
    asm volatile("ld.shared.v2.f32 {%0, %1}, [%2];" : "=f"(a), "=f"(b) : "r"(addr) : "memory");
}
// Start-up rendezvous of a cluster: no data is handed over (mbarrier initialisation is published
// by fence.mbarrier_init), so the arrive carries no memory fence.
__device__ __forceinline__ void cluster_arrive_relaxed() {
    asm volatile("barrier.cluster.arrive.relaxed.aligned;" ::: "memory");
}
__device__ __forceinline__ void cluster_wait_acquire() {
    asm volatile("barrier.cluster.wait.acquire.aligned;" ::: "memory");
}

}  // namespace fsm
