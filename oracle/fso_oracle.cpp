// fso_oracle.cpp -- TEST INFRASTRUCTURE, not part of the product.
//
// Plain, slow, single-threaded fp64 statement of the last-dimension softmax
//     y_ij = exp(z_ij - max_k z_ik) / sum_k exp(z_ik - max_k z_ik),   z = scale * x,
// the operator the paper names in its abstract and in Sec. IV-C (Gemma 4 E2B / Qwen 3.5
// softmax results). The paper's Sec. III-C ("Kernel Validator") defines correctness as
// agreement with the eager framework output on the same inputs within a per-dtype
// tolerance; this file is that reference, written from the definition, and the
// comparator that applies the tolerance.
//
// Only tests, the smoke check and the benchmark's cpu_baseline leg may call this file.
// It shares no code, header, table or constant with the CUDA library.
//
// Every function here is pinned by tests that do not call it to produce their expected
// values (closed forms, 100-digit mpmath evaluation, brute force on tiny rows, exhaustive
// 16-bit round trips): nothing is "parity unpinned".
//
// Build: g++ -O2 -std=c++17 -ffp-contract=off -fno-fast-math -shared -fPIC

#include <cmath>
#include <cstdint>
#include <cstring>
#include <limits>

namespace {

enum { DT_FP32 = 0, DT_BF16 = 1, DT_FP16 = 2 };

// ---- exact widening of one stored element to double ------------------------------------

double widen_fp32(const void* p, int64_t i) {
    float f;
    std::memcpy(&f, static_cast<const char*>(p) + 4 * i, 4);
    return static_cast<double>(f);
}

// bfloat16 is the upper half of an IEEE binary32 pattern.
double widen_bf16(const void* p, int64_t i) {
    uint16_t h;
    std::memcpy(&h, static_cast<const char*>(p) + 2 * i, 2);
    uint32_t w = static_cast<uint32_t>(h) << 16;
    float f;
    std::memcpy(&f, &w, 4);
    return static_cast<double>(f);
}

// IEEE binary16: 1 sign, 5 exponent (bias 15), 10 fraction bits.
double widen_fp16(const void* p, int64_t i) {
    uint16_t h;
    std::memcpy(&h, static_cast<const char*>(p) + 2 * i, 2);
    const int sign = h >> 15;
    const int expo = (h >> 10) & 0x1f;
    const int frac = h & 0x3ff;
    double v;
    if (expo == 0x1f) {
        v = frac ? std::numeric_limits<double>::quiet_NaN()
                 : std::numeric_limits<double>::infinity();
    } else if (expo == 0) {
        v = std::ldexp(static_cast<double>(frac), -24);          // subnormal: frac * 2^-24
    } else {
        v = std::ldexp(static_cast<double>(1024 + frac), expo - 25);  // (1 + frac/1024) * 2^(expo-15)
    }
    return sign ? -v : v;
}

double widen(const void* p, int dtype, int64_t i) {
    switch (dtype) {
        case DT_FP32: return widen_fp32(p, i);
        case DT_BF16: return widen_bf16(p, i);
        default:      return widen_fp16(p, i);
    }
}

// ---- direct round-to-nearest-even of a double to a 16-bit format -----------------------
// Works on the value, not through float, so there is no double rounding.
// fmt_frac = stored fraction bits (7 for bfloat16, 10 for binary16),
// emin = exponent of the smallest normal, emax = exponent of the largest finite binade.

uint16_t round_to_16(double v, int fmt_frac, int emin, int emax, int expo_bits) {
    const uint16_t sign = std::signbit(v) ? 0x8000u : 0u;
    const int bias = -emin + 1;
    const uint16_t expo_all = static_cast<uint16_t>(((1u << expo_bits) - 1u) << fmt_frac);
    if (std::isnan(v)) return static_cast<uint16_t>(sign | expo_all | (1u << (fmt_frac - 1)));
    double a = std::fabs(v);
    if (std::isinf(a)) return static_cast<uint16_t>(sign | expo_all);
    if (a == 0.0) return sign;
    int e;
    std::frexp(a, &e);            // a = m * 2^e, m in [0.5, 1)  ->  binade exponent e-1
    int binade = e - 1;
    if (binade < emin) binade = emin;                 // subnormal range shares emin's spacing
    // spacing of representable values in this binade: 2^(binade - fmt_frac)
    const double q = std::ldexp(a, fmt_frac - binade);  // exact scaling by a power of two
    const double n = std::nearbyint(q);                 // default rounding mode: ties to even
    // n is an integer in [0, 2^(fmt_frac+1)]; rebuild the pattern arithmetically so that a
    // carry out of the fraction moves into the exponent field by itself.
    int64_t ni = static_cast<int64_t>(n);
    int64_t pattern;
    if (binade == emin && ni < (int64_t(1) << fmt_frac)) {
        pattern = ni;                                                    // subnormal or zero
    } else {
        pattern = (static_cast<int64_t>(binade + bias) << fmt_frac) + (ni - (int64_t(1) << fmt_frac));
    }
    const int64_t inf_pattern = static_cast<int64_t>(expo_all);
    if (pattern >= inf_pattern || binade > emax) pattern = inf_pattern;  // overflow -> inf
    return static_cast<uint16_t>(sign | static_cast<uint16_t>(pattern));
}

uint16_t round_bf16(double v) { return round_to_16(v, 7, -126, 127, 8); }
uint16_t round_fp16(double v) { return round_to_16(v, 10, -14, 15, 5); }

// Signed ordinal of a 16-bit sign-magnitude pattern: neighbours differ by one.
int32_t ordinal16(uint16_t b) {
    const int32_t mag = b & 0x7fff;
    return (b & 0x8000) ? -mag : mag;
}

bool is_nan16(uint16_t b, int dtype) {
    if (dtype == DT_BF16) return (b & 0x7f80) == 0x7f80 && (b & 0x007f) != 0;
    return (b & 0x7c00) == 0x7c00 && (b & 0x03ff) != 0;
}

}  // namespace

extern "C" {

// One row of the definition. x: `cols` stored elements of `dtype`; y: `cols` doubles.
// Steps, in the order of the formula:
//   z_j = scale * x_j         (exact in fp64: two <=24-bit significands)
//   M   = max_j z_j           (left-to-right scan)
//   e_j = exp(z_j - M)
//   S   = sum_j e_j           (left to right, Neumaier-compensated)
//   y_j = e_j / S
// IEEE special values are evaluated literally: a NaN or +inf anywhere, or a row of only
// -inf, makes S NaN and so the whole row NaN; a -inf beside finite entries gives exactly +0.
void fso_softmax_row_f64(const void* x, int dtype, int64_t cols, float scale, double* y) {
    if (cols <= 0) return;
    const double sc = static_cast<double>(scale);
    for (int64_t j = 0; j < cols; ++j) y[j] = sc * widen(x, dtype, j);   // y holds z for now
    double M = y[0];
    for (int64_t j = 1; j < cols; ++j) {
        if (y[j] > M) M = y[j];
    }
    double S = 0.0, comp = 0.0;
    for (int64_t j = 0; j < cols; ++j) {
        const double e = std::exp(y[j] - M);
        y[j] = e;
        const double t = S + e;
        if (std::fabs(S) >= std::fabs(e)) comp += (S - t) + e;
        else                              comp += (e - t) + S;
        S = t;
    }
    S += comp;
    for (int64_t j = 0; j < cols; ++j) y[j] = y[j] / S;
}

// Whole matrix, row after row. x: rows*cols stored elements, row-major; y: rows*cols doubles.
void fso_softmax_f64(const void* x, int dtype, int64_t rows, int64_t cols, float scale, double* y) {
    const int64_t esz = (dtype == DT_FP32) ? 4 : 2;
    for (int64_t i = 0; i < rows; ++i) {
        fso_softmax_row_f64(static_cast<const char*>(x) + i * cols * esz, dtype, cols, scale, y + i * cols);
    }
}

// log_softmax, the logarithm of the same operator (the form language-model heads consume; the
// paper's harness captures softmax-family operators per model, Sec. III-A):
//   z_j = scale * x_j;  M = max_j z_j;  S = sum_j exp(z_j - M) (Neumaier);  y_j = (z_j - M) - log(S)
// A -inf entry beside finite ones gives -inf; a NaN or +inf entry, or a row of only -inf, makes
// the whole row NaN, as for the softmax.
void fso_log_softmax_f64(const void* x, int dtype, int64_t rows, int64_t cols, float scale, double* y) {
    const int64_t esz = (dtype == DT_FP32) ? 4 : 2;
    const double sc = static_cast<double>(scale);
    for (int64_t i = 0; i < rows; ++i) {
        const void* xr = static_cast<const char*>(x) + i * cols * esz;
        double* yr = y + i * cols;
        if (cols <= 0) continue;
        for (int64_t j = 0; j < cols; ++j) yr[j] = sc * widen(xr, dtype, j);
        double M = yr[0];
        for (int64_t j = 1; j < cols; ++j) {
            if (yr[j] > M) M = yr[j];
        }
        double S = 0.0, comp = 0.0;
        for (int64_t j = 0; j < cols; ++j) {
            const double e = std::exp(yr[j] - M);
            const double t = S + e;
            if (std::fabs(S) >= std::fabs(e)) comp += (S - t) + e;
            else                              comp += (e - t) + S;
            S = t;
        }
        S += comp;
        const double L = std::log(S);
        for (int64_t j = 0; j < cols; ++j) yr[j] = (yr[j] - M) - L;
    }
}

// Additive-mask variant (the `scores + mask` that eager attention forms before its softmax; fusing
// the addition is the operator-fusion lever of the paper's Sec. II-B):
//   z_ij = scale * x_ij + mask[mrow(i)][j],   y_i = softmax(z_i)
// x: rows ordered (batch, head, query); the mask has one row per (batch, query) and is shared by the
// heads: mrow(i) = (i / (heads * q_rows)) * q_rows + i % q_rows. The mask is not scaled.
void fso_softmax_masked_f64(const void* x, const void* mask, int dtype, int64_t rows, int64_t cols, int64_t q_rows,
                            int64_t heads, float scale, double* y) {
    const int64_t esz = (dtype == DT_FP32) ? 4 : 2;
    const double sc = static_cast<double>(scale);
    for (int64_t i = 0; i < rows; ++i) {
        const void* xr = static_cast<const char*>(x) + i * cols * esz;
        const int64_t mrow = (i / (heads * q_rows)) * q_rows + i % q_rows;
        const void* mr = static_cast<const char*>(mask) + mrow * cols * esz;
        double* yr = y + i * cols;
        if (cols <= 0) continue;
        for (int64_t j = 0; j < cols; ++j) yr[j] = sc * widen(xr, dtype, j) + widen(mr, dtype, j);
        double M = yr[0];
        for (int64_t j = 1; j < cols; ++j) {
            if (yr[j] > M) M = yr[j];
        }
        double S = 0.0, comp = 0.0;
        for (int64_t j = 0; j < cols; ++j) {
            const double e = std::exp(yr[j] - M);
            yr[j] = e;
            const double t = S + e;
            if (std::fabs(S) >= std::fabs(e)) comp += (S - t) + e;
            else                              comp += (e - t) + S;
            S = t;
        }
        S += comp;
        for (int64_t j = 0; j < cols; ++j) yr[j] = yr[j] / S;
    }
}

// Backward of y = softmax(scale * x) (the gradient a training step needs from the same operator):
//   dx_j = scale * y_j * (dy_j - sum_k dy_k y_k)
// dy, y: stored elements of `dtype`; dx: doubles. The dot product is a left-to-right Neumaier sum.
void fso_softmax_backward_f64(const void* dy, const void* y, int dtype, int64_t rows, int64_t cols, float scale, double* dx) {
    const int64_t esz = (dtype == DT_FP32) ? 4 : 2;
    const double sc = static_cast<double>(scale);
    for (int64_t i = 0; i < rows; ++i) {
        const void* gr = static_cast<const char*>(dy) + i * cols * esz;
        const void* yr = static_cast<const char*>(y) + i * cols * esz;
        double S = 0.0, comp = 0.0;
        for (int64_t j = 0; j < cols; ++j) {
            const double e = widen(gr, dtype, j) * widen(yr, dtype, j);
            const double t = S + e;
            if (std::fabs(S) >= std::fabs(e)) comp += (S - t) + e;
            else                              comp += (e - t) + S;
            S = t;
        }
        S += comp;
        for (int64_t j = 0; j < cols; ++j) dx[i * cols + j] = sc * (widen(yr, dtype, j) * (widen(gr, dtype, j) - S));
    }
}

// Causal variant (the mask eager attention applies before its softmax; fusing it is the "operator
// fusion" lever of the paper's Sec. II-B): row i keeps columns j <= i + q_offset and the softmax is
// taken over the kept columns only; a masked column has z = -inf, i.e. y = exactly +0, whatever is
// stored there (it is never read). A row with no kept column is all NaN, like any row whose
// entries are all -inf; a row that a kept NaN or +inf makes NaN is NaN in its masked part too.
void fso_softmax_causal_f64(const void* x, int dtype, int64_t rows, int64_t cols, int64_t q_offset,
                            float scale, double* y) {
    const int64_t esz = (dtype == DT_FP32) ? 4 : 2;
    for (int64_t i = 0; i < rows; ++i) {
        int64_t keep = i + q_offset + 1;                  // number of leading columns kept
        if (keep < 0) keep = 0;
        if (keep > cols) keep = cols;
        double* yr = y + i * cols;
        if (keep == 0) {
            for (int64_t j = 0; j < cols; ++j) yr[j] = std::numeric_limits<double>::quiet_NaN();
            continue;
        }
        fso_softmax_row_f64(static_cast<const char*>(x) + i * cols * esz, dtype, keep, scale, yr);
        // literally 0 / S: +0, or NaN when a kept NaN or +inf has made the row NaN
        for (int64_t j = keep; j < cols; ++j) yr[j] = 0.0 * yr[0];
    }
}

// Router step of a mixture-of-experts layer (the softmax over expert logits of the paper's
// Qwen 3.5 35B-A3B workload, Table I, followed by the selection every such router makes):
//   p = softmax(scale * x_row);  take the k largest p, ties going to the lower column;
//   w_j = p[idx_j], or p[idx_j] / sum of the k selected p when `renorm` is set.
// The order of p is the order of z = scale * x (exp is increasing), and z is exact in fp64, so
// the selection is made on z: a stable sort by decreasing z, a NaN z counting as -inf.
// w: rows*k doubles, idx: rows*k int32, both in selection order (largest first).
void fso_router_topk_f64(const void* x, int dtype, int64_t rows, int64_t cols, int64_t k, float scale,
                         int renorm, double* w, int32_t* idx) {
    const int64_t esz = (dtype == DT_FP32) ? 4 : 2;
    const double sc = static_cast<double>(scale);
    double* p = new double[static_cast<size_t>(cols > 0 ? cols : 1)];
    double* key = new double[static_cast<size_t>(cols > 0 ? cols : 1)];
    int32_t* order = new int32_t[static_cast<size_t>(cols > 0 ? cols : 1)];
    for (int64_t i = 0; i < rows; ++i) {
        const char* row = static_cast<const char*>(x) + i * cols * esz;
        fso_softmax_row_f64(row, dtype, cols, scale, p);
        for (int64_t j = 0; j < cols; ++j) {
            const double z = sc * widen(row, dtype, j);
            key[j] = std::isnan(z) ? -std::numeric_limits<double>::infinity() : z;
            order[j] = static_cast<int32_t>(j);
        }
        // stable insertion sort by decreasing key (plain and obviously stable; cols is small)
        for (int64_t a = 1; a < cols; ++a) {
            const int32_t cur = order[a];
            int64_t b = a;
            while (b > 0 && key[order[b - 1]] < key[cur]) { order[b] = order[b - 1]; --b; }
            order[b] = cur;
        }
        double sel = 0.0;
        for (int64_t j = 0; j < k; ++j) sel += p[order[j]];
        for (int64_t j = 0; j < k; ++j) {
            idx[i * k + j] = order[j];
            w[i * k + j] = renorm ? p[order[j]] / sel : p[order[j]];
        }
    }
    delete[] p; delete[] key; delete[] order;
}

// Exact widening of stored elements (exposed so tests can pin the decoders).
void fso_widen(const void* x, int dtype, int64_t n, double* out) {
    for (int64_t i = 0; i < n; ++i) out[i] = widen(x, dtype, i);
}

// Round doubles to the stored format, nearest-even, directly from fp64.
// dtype fp32 uses the hardware double->float conversion (one rounding by IEEE rules).
void fso_round_from_f64(const double* v, int dtype, int64_t n, void* out) {
    for (int64_t i = 0; i < n; ++i) {
        if (dtype == DT_FP32) {
            const float f = static_cast<float>(v[i]);
            std::memcpy(static_cast<char*>(out) + 4 * i, &f, 4);
        } else {
            const uint16_t b = (dtype == DT_BF16) ? round_bf16(v[i]) : round_fp16(v[i]);
            std::memcpy(static_cast<char*>(out) + 2 * i, &b, 2);
        }
    }
}

struct fso_report {
    double  max_abs_err;     // fp32: max |got - want| over comparable elements (0 for 16-bit)
    int64_t max_ulp;         // 16-bit: max |ord(got) - ord(RN(want))| (0 for fp32)
    int64_t nan_mismatch;    // want NaN xor got NaN
    int64_t zero_mismatch;   // want is exactly +0 but got's bit pattern is not +0
    int64_t negative;        // got has its sign bit set with a non-zero magnitude (softmax is >= 0)
    int64_t worst_index;     // element where max_abs_err / max_ulp was reached (-1 if none)
    int64_t n_compared;
};

// Compare a device result (`got`, stored dtype) with the oracle's fp64 values (`want`).
//   fp32 : error = |(double)got - want| against the unrounded fp64 value.
//   16-bit: distance in units of the last place between got and the fp64 value rounded
//           once, nearest-even, to the format (subnormal spacing in the subnormal range).
//   NaN matches any NaN. An oracle value that is exactly +0 (a -inf input, or an fp64
//   underflow) must be matched by the +0 bit pattern.
void fso_compare(const void* got, int dtype, const double* want, int64_t n, fso_report* rep) {
    fso_report r{};
    r.worst_index = -1;
    for (int64_t i = 0; i < n; ++i) {
        const double w = want[i];
        if (dtype == DT_FP32) {
            float g;
            std::memcpy(&g, static_cast<const char*>(got) + 4 * i, 4);
            const bool gn = std::isnan(g), wn = std::isnan(w);
            if (gn || wn) { if (gn != wn) ++r.nan_mismatch; continue; }
            uint32_t gb; std::memcpy(&gb, &g, 4);
            if (w == 0.0 && gb != 0u) ++r.zero_mismatch;
            if (std::signbit(g) && g != 0.0f) ++r.negative;
            const double err = std::fabs(static_cast<double>(g) - w);
            if (err > r.max_abs_err || r.worst_index < 0) {
                r.worst_index = i;
                if (err > r.max_abs_err) r.max_abs_err = err;
            }
        } else {
            uint16_t g;
            std::memcpy(&g, static_cast<const char*>(got) + 2 * i, 2);
            const bool gn = is_nan16(g, dtype), wn = std::isnan(w);
            if (gn || wn) { if (gn != wn) ++r.nan_mismatch; continue; }
            if (w == 0.0 && g != 0u) ++r.zero_mismatch;
            if ((g & 0x8000) && (g & 0x7fff)) ++r.negative;
            const uint16_t wr = (dtype == DT_BF16) ? round_bf16(w) : round_fp16(w);
            int64_t d = static_cast<int64_t>(ordinal16(g)) - static_cast<int64_t>(ordinal16(wr));
            if (d < 0) d = -d;
            if (d > r.max_ulp || r.worst_index < 0) {
                r.worst_index = i;
                if (d > r.max_ulp) r.max_ulp = d;
            }
        }
        ++r.n_compared;
    }
    *rep = r;
}

}  // extern "C"
