// CPU oracle for the H-BitLinear forward pass (BitNet v2, section 2.1).
//
// TEST INFRASTRUCTURE, not product: a plain, slow, step-by-step restatement of
// the paper's definitions (Eq. 1-7: absmean ternary weights, the Sylvester
// Hadamard recursion, per-token absmax-INT8 / absmean-INT4 activation
// quantizers, the integer contraction and the rescale; plus the normalisation and
// gating product that feed the layer and the low-bit attention-state quantizer of
// section 3.1, each marked where it is defined).  It shares no code with
// the CUDA path and must only be used by the tests, the smoke check and the
// benchmark's CPU-baseline leg.
//
// Arithmetic: fp64 throughout, with one rounding at each point that the layer's
// storage types force (alpha -> fp32, scales -> fp32 on output, y -> bf16).  The
// one place where floating point decides an integer -- round(W/(alpha+eps)) and
// round(c*x/(stat+eps)) -- can be taken either in fp64 (`prec == 64`) or in the
// kernel's precision, IEEE fp32 with the operations in the order the formulas
// are written (`prec == 32`), so that both sides of a parity test take that
// decision in the same precision.
//
// Readings the paper leaves open (fixed here, stated in the design notes):
// round() is round-half-to-even; eps is an explicit argument and appears in the
// quantizing division only, never in the dequantizing scale; the transform is
// orthonormal (1/sqrt(2) per level => 1/sqrt(n) overall), natural (Sylvester)
// order, over the whole in_dim of each token; per-token statistics are taken
// over the post-transform vector.  Parity unpinned: the value of eps and the
// tie rule of round() -- nothing the paper prints fixes them.
//
// Parallel over tokens / rows only (OpenMP); no blocking, no fusion.

#include <cmath>
#include <cstdint>
#include <cstdlib>
#include <cstring>
#include <vector>
#ifdef _OPENMP
#include <omp.h>
#endif

namespace {

inline double round_half_even(double v) { return std::nearbyint(v); }   // default FE_TONEAREST
inline float round_half_even_f(float v) { return std::nearbyintf(v); }

inline double clipd(double v, double lo, double hi) { return std::fmin(std::fmax(v, lo), hi); }

// bf16 bits of a double, one rounding (nearest even) from the exact value.
// Done through fp32 only when that is exact: a double product is first rounded
// to the 8-bit significand directly to avoid double rounding.
inline uint16_t bf16_from_double(double v) {
    if (std::isnan(v)) return 0x7FC0;
    if (v == 0.0) return std::signbit(v) ? 0x8000 : 0x0000;
    if (std::isinf(v)) return std::signbit(v) ? 0xFF80 : 0x7F80;
    int e;
    double m = std::frexp(std::fabs(v), &e);          // |v| = m * 2^e, m in [0.5,1)
    int exp_unb = e - 1;                               // |v| = (2m) * 2^(e-1), 2m in [1,2)
    if (exp_unb < -126) {                              // bf16 subnormal range: spacing 2^-133
        double q = std::nearbyint(std::ldexp(std::fabs(v), 133));
        uint32_t mant = (uint32_t)q;                   // may reach 128 => smallest normal
        uint16_t bits = (uint16_t)mant;                // exponent field 0 (or carries into 1)
        return (uint16_t)(bits | (std::signbit(v) ? 0x8000 : 0));
    }
    double sig = std::nearbyint(std::ldexp(m, 8));     // 8-bit significand in [128,256]
    if (sig >= 256.0) { sig = 128.0; exp_unb += 1; }
    if (exp_unb > 127) return std::signbit(v) ? 0xFF80 : 0x7F80;
    uint32_t bits = ((uint32_t)(exp_unb + 127) << 7) | ((uint32_t)sig & 0x7F);
    return (uint16_t)(bits | (std::signbit(v) ? 0x8000 : 0));
}

}  // namespace

extern "C" {

int orc_num_threads() {
#ifdef _OPENMP
    return omp_get_max_threads();
#else
    return 1;
#endif
}

// Eq. 1-2.  alpha = mean(|W|) over the whole tensor; W_t = RoundClip(W/(alpha+eps), -1, 1).
// W: fp32 [N,K] row-major.  wt: int8 [N,K].  alpha_out: the fp32 alpha that is stored.
int orc_weight_quant(const float* W, long N, long K, float eps, int prec,
                     int8_t* wt, float* alpha_out) {
    const long total = N * K;
    if (total <= 0) return 1;
    // fp64 sum, row by row then over rows: error ~1e-16 relative, far below fp32.
    std::vector<double> rowsum((size_t)N, 0.0);
#pragma omp parallel for schedule(static)
    for (long o = 0; o < N; ++o) {
        double s = 0.0;
        for (long k = 0; k < K; ++k) s += std::fabs((double)W[o * K + k]);
        rowsum[(size_t)o] = s;
    }
    double s = 0.0;
    for (long o = 0; o < N; ++o) s += rowsum[(size_t)o];
    const float alpha = (float)(s / (double)total);
    *alpha_out = alpha;
    if (prec == 32) {
        const float d = alpha + eps;
#pragma omp parallel for schedule(static)
        for (long i = 0; i < total; ++i) {
            float r = round_half_even_f(W[i] / d);
            wt[i] = (int8_t)std::fmin(std::fmax(r, -1.0f), 1.0f);
        }
    } else {
        const double d = (double)alpha + (double)eps;
#pragma omp parallel for schedule(static)
        for (long i = 0; i < total; ++i)
            wt[i] = (int8_t)clipd(round_half_even((double)W[i] / d), -1.0, 1.0);
    }
    return 0;
}

// Eq. 3-4.  x_r = H_m x for every token (row), H_m the orthonormal Sylvester matrix:
// the recursion H_m = 1/sqrt(2) [[H,H],[H,-H]] unrolled level by level into
// butterflies (a,b) -> (a+b, a-b) on index pairs (i, i+h), h = 1,2,4,...; the
// m factors of 1/sqrt(2) are applied once as 1/sqrt(n).
// x: fp32 [T,K]; xr: fp64 [T,K].  K must be a power of two.
int orc_hadamard(const float* x, long T, long K, double* xr) {
    if (K <= 0 || (K & (K - 1)) != 0) return 3;
    const double norm = 1.0 / std::sqrt((double)K);
#pragma omp parallel for schedule(static)
    for (long t = 0; t < T; ++t) {
        double* v = xr + t * K;
        for (long k = 0; k < K; ++k) v[k] = (double)x[t * K + k];
        for (long h = 1; h < K; h *= 2)
            for (long base = 0; base < K; base += 2 * h)
                for (long i = base; i < base + h; ++i) {
                    double a = v[i], b = v[i + h];
                    v[i] = a + b;
                    v[i + h] = a - b;
                }
        for (long k = 0; k < K; ++k) v[k] *= norm;
    }
    return 0;
}

// No transform: widen the token to fp64 unchanged (the plain BitLinear input).
int orc_widen(const float* x, long T, long K, double* xr) {
    for (long i = 0; i < T * K; ++i) xr[i] = (double)x[i];
    return 0;
}

// Eq. 5 (bits == 8): gamma = max|x|, q = RoundClip(127/(gamma+eps) * x, -128, 127), s = gamma/127.
// Eq. 6 (bits == 4): beta = mean|x|, q = RoundClip(sqrt(7)/(beta+eps) * x, -8, 7),  s = beta/sqrt(7).
// xr: fp64 [T,K] (the vector that is quantized: post-transform when the layer
// transforms).  Outputs per token: codes q (int8), pre-rounding values v (fp64,
// may be null), dequantization scale s (fp64) and the statistic (fp64, may be null).
// prec == 32 takes stat -> fp32, then d = stat+eps, r = c/d, v = r*x in IEEE fp32.
int orc_act_quant(const double* xr, long T, long K, int bits, float eps, int prec,
                  int8_t* q, double* v_out, double* s_out, double* stat_out) {
    if (bits != 4 && bits != 8) return 4;
    const double c = (bits == 8) ? 127.0 : std::sqrt(7.0);
    const double lo = (bits == 8) ? -128.0 : -8.0;
    const double hi = (bits == 8) ? 127.0 : 7.0;
#pragma omp parallel for schedule(static)
    for (long t = 0; t < T; ++t) {
        const double* x = xr + t * K;
        double stat = 0.0;
        if (bits == 8) {
            for (long k = 0; k < K; ++k) stat = std::fmax(stat, std::fabs(x[k]));
        } else {
            for (long k = 0; k < K; ++k) stat += std::fabs(x[k]);
            stat /= (double)K;
        }
        if (prec == 32) {
            const float stat32 = (float)stat;
            const float r = (float)c / (stat32 + eps);
            for (long k = 0; k < K; ++k) {
                const float v = r * (float)x[k];
                if (v_out) v_out[t * K + k] = (double)v;
                q[t * K + k] = (int8_t)std::fmin(std::fmax(round_half_even_f(v), (float)lo), (float)hi);
            }
            s_out[t] = (double)stat32 / c;
            if (stat_out) stat_out[t] = (double)stat32;
        } else {
            const double r = c / (stat + (double)eps);
            for (long k = 0; k < K; ++k) {
                const double v = r * x[k];
                if (v_out) v_out[t * K + k] = v;
                q[t * K + k] = (int8_t)clipd(round_half_even(v), lo, hi);
            }
            s_out[t] = stat / c;
            if (stat_out) stat_out[t] = stat;
        }
    }
    return 0;
}

// Eq. 7, the contraction: acc[t,o] = sum_k wt[o,k] * q[t,k], exact integers.
// Accumulated in int64 and checked to fit int32.  Returns 20 on overflow.
int orc_gemm(const int8_t* q, const int8_t* wt, long T, long K, long N, int32_t* acc) {
    int bad = 0;
#pragma omp parallel for schedule(static) reduction(| : bad)
    for (long t = 0; t < T; ++t)
        for (long o = 0; o < N; ++o) {
            int64_t a = 0;
            for (long k = 0; k < K; ++k) a += (int64_t)wt[o * K + k] * (int64_t)q[t * K + k];
            if (a > INT32_MAX || a < INT32_MIN) bad |= 1;
            acc[t * N + o] = (int32_t)a;
        }
    return bad ? 20 : 0;
}

// The normalisation in front of the transform ("LN" in Eq. 7; section 2 builds the model from RMS
// normalisation, no biases): out[t,k] = x[t,k] / sqrt(mean_k x[t,k]^2 + eps_ln) * g[k], computed in
// fp64 and rounded once to bf16, the type activations are stored in (returned widened to fp32, every
// value exactly a bf16).  pre (may be null): the fp64 values before that rounding.
// Reading taken where the paper is silent: RMS normalisation (no mean subtraction), a learned gain
// vector, eps_ln inside the square root, result in bf16.  Parity unpinned for those choices.
int orc_rmsnorm_bf16(const float* x, const float* g, long T, long K, float eps_ln, float* out, double* pre) {
    if (T < 0 || K <= 0 || eps_ln < 0.0f) return 30;
#pragma omp parallel for schedule(static)
    for (long t = 0; t < T; ++t) {
        double ss = 0.0;
        for (long k = 0; k < K; ++k) ss += (double)x[t * K + k] * (double)x[t * K + k];
        const double rms = std::sqrt(ss / (double)K + (double)eps_ln);
        for (long k = 0; k < K; ++k) {
            const double v = rms > 0.0 ? (double)x[t * K + k] / rms * (double)g[k] : 0.0;
            if (pre) pre[t * K + k] = v;
            const uint32_t bits = (uint32_t)bf16_from_double(v) << 16;
            float f;
            std::memcpy(&f, &bits, 4);
            out[t * K + k] = f;
        }
    }
    return 0;
}

// The input of W_down in a SwishGLU feed-forward block (section 2 names SwishGLU among the model's
// components): out[t,k] = SiLU(gate[t,k]) * up[t,k] with SiLU(z) = z / (1 + exp(-z)), computed in fp64
// and rounded once to bf16 (returned widened to fp32).  pre (may be null): the fp64 values before that
// rounding.  Reading taken where the paper is silent: which projection passes through SiLU (the one
// called gate here), and bf16 as the type of the product.  Parity unpinned for those choices.
int orc_swiglu_bf16(const float* gate, const float* up, long T, long K, float* out, double* pre) {
    if (T < 0 || K <= 0) return 31;
#pragma omp parallel for schedule(static)
    for (long i = 0; i < T * K; ++i) {
        const double z = (double)gate[i];
        const double v = z / (1.0 + std::exp(-z)) * (double)up[i];
        if (pre) pre[i] = v;
        const uint32_t bits = (uint32_t)bf16_from_double(v) << 16;
        float f;
        std::memcpy(&f, &bits, 4);
        out[i] = f;
    }
    return 0;
}

// Eq. 1, 5-7, the prefactors: y[t,o] = alpha * s_t * acc[t,o], rounded once to bf16.
// y_bits: bf16 bit patterns [T,N]; y64 (may be null): the unrounded fp64 values.
int orc_rescale(const int32_t* acc, const double* s, float alpha, long T, long N,
                uint16_t* y_bits, double* y64) {
#pragma omp parallel for schedule(static)
    for (long t = 0; t < T; ++t)
        for (long o = 0; o < N; ++o) {
            const double y = (double)acc[t * N + o] * s[t] * (double)alpha;
            if (y64) y64[t * N + o] = y;
            y_bits[t * N + o] = bf16_from_double(y);
        }
    return 0;
}

// Low-bit attention states (section 3.1, Tables 2-3): the Q, K and V heads are quantized after the rotary
// embedding "to unsigned integers using the absmax function", and the K/V heads of the [BOS] token stay at
// 8 bits.  The paper prints no formula; the reading taken is Eq. 5's absmax quantizer at b bits, one
// statistic per head of each token, stored with an offset so that the code is unsigned:
//     gamma = max_d |x[d]|,   q = RoundClip((2^(b-1) - 1) / (gamma + eps) * x, -2^(b-1), 2^(b-1) - 1),
//     u = q + 2^(b-1)  in [0, 2^b - 1],   dequantization scale s = gamma / (2^(b-1) - 1).
// (b = 8 is Eq. 5 itself plus the offset 128.)  Every choice here -- per-head granularity, the symmetric
// grid, the offset -- is a reading: parity unpinned.
// x: fp32 [R, D] (R = tokens * heads rows of one head each).  bits_row (may be null): bits per row, for the
// rows kept at another width (the [BOS] token's heads at 8); otherwise `bits` for every row.
// Outputs: u (uint8, one code per byte), v (fp64 pre-rounding values, may be null), s (fp64 [R]).
int orc_kv_quant(const float* x, long R, long D, int bits, const int* bits_row, float eps, int prec,
                 uint8_t* u, double* v_out, double* s_out) {
    if (bits < 2 || bits > 8) return 4;
    int bad = 0;
#pragma omp parallel for schedule(static) reduction(| : bad)
    for (long r = 0; r < R; ++r) {
        const int b = bits_row ? bits_row[r] : bits;
        if (b < 2 || b > 8) { bad |= 1; continue; }
        const double half = (double)(1 << (b - 1));            // 2^(b-1)
        const double c = half - 1.0;
        const float* row = x + r * D;
        double gamma = 0.0;
        for (long d = 0; d < D; ++d) gamma = std::fmax(gamma, std::fabs((double)row[d]));
        if (prec == 32) {
            const float g32 = (float)gamma;
            const float rq = (float)c / (g32 + eps);
            for (long d = 0; d < D; ++d) {
                const float v = rq * row[d];
                if (v_out) v_out[r * D + d] = (double)v;
                const float q = std::fmin(std::fmax(round_half_even_f(v), (float)-half), (float)(half - 1.0));
                u[r * D + d] = (uint8_t)((int)q + (int)half);
            }
            s_out[r] = (double)g32 / c;
        } else {
            const double rq = c / (gamma + (double)eps);
            for (long d = 0; d < D; ++d) {
                const double v = rq * (double)row[d];
                if (v_out) v_out[r * D + d] = v;
                u[r * D + d] = (uint8_t)((int)clipd(round_half_even(v), -half, half - 1.0) + (int)half);
            }
            s_out[r] = gamma / c;
        }
    }
    return bad ? 4 : 0;
}

// The whole layer for T tokens against already-ternarised weights: Eq. 3-7 chained.
// Scratch is allocated here; outputs as in the stage functions (codes/acc may be null).
int orc_forward(const float* x, long T, long K, const int8_t* wt, float alpha, long N,
                int bits, int use_hadamard, float eps, int prec,
                uint16_t* y_bits, double* y64, int8_t* codes_out, int32_t* acc_out,
                double* s_out) {
    std::vector<double> xr((size_t)(T * K));
    std::vector<int8_t> q((size_t)(T * K));
    std::vector<double> s((size_t)T);
    std::vector<int32_t> acc((size_t)(T * N));
    int rc = use_hadamard ? orc_hadamard(x, T, K, xr.data()) : orc_widen(x, T, K, xr.data());
    if (rc) return rc;
    rc = orc_act_quant(xr.data(), T, K, bits, eps, prec, q.data(), nullptr, s.data(), nullptr);
    if (rc) return rc;
    rc = orc_gemm(q.data(), wt, T, K, N, acc.data());
    if (rc) return rc;
    rc = orc_rescale(acc.data(), s.data(), alpha, T, N, y_bits, y64);
    if (codes_out) std::memcpy(codes_out, q.data(), (size_t)(T * K));
    if (acc_out) std::memcpy(acc_out, acc.data(), sizeof(int32_t) * (size_t)(T * N));
    if (s_out) std::memcpy(s_out, s.data(), sizeof(double) * (size_t)T);
    return rc;
}

}  // extern "C"
