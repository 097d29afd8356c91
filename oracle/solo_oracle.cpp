// SOLO low-bit optimizer step -- CPU oracle (TEST INFRASTRUCTURE, not the product).
//
// A plain, slow, scalar restatement of what the paper "Pushing the Limits of
// Low-Bit Optimizers: A Focus on EMA Dynamics" (SOLO) defines for one
// optimizer step on block-wise quantized Adam(W) states.  It exists so that the
// CUDA library can be checked against something written independently from the
// paper; it shares no code, header, table or constant generator with that
// library.  Only tests, the smoke check and the benchmark's CPU-baseline leg may
// load it; the product never does.
//
// Precision: every quantity that decides a stored integer code (the EMA values,
// the block scales, the quantile, the logarithm that is rounded) is computed in
// IEEE binary32 with round-to-nearest, one rounding per written operation
// (compile with -ffp-contract=off; fused multiply-adds are written out as
// std::fmaf).  That is the precision the kernel works in; the decision is taken
// in the same precision on both sides.  Scalars that depend only on the
// hyper-parameters (bias corrections) are computed in binary64 and rounded once.
//
// Pins (see tests/test_oracle_*.py): codebooks vs Fact A.1 radii, Corollary 3.2
// thresholds, the beta' table of Eq. 7 (Fig. 4), Theorem 3.1 as a property,
// Proposition 3.5 decay statistics, Theorem 3.6 (unbiased SR, variance bound),
// brute-force nearest-level search, Philox known answers, textbook AdamW,
// memory accounting of Table 2, the stochastic bf16 rounding over all 2^16
// draws, the baseline second-moment codebooks by exhaustive search, the
// swamping of Corollary 3.2 through the whole step, the decode of the previous
// packed state (Eq. 2) redone in binary64 from the bytes with the Appendix A
// levels typed out, and every Eq. 5 code of the step against the element's own
// draw.  Unpinned (paper silent; internal consistency
// only): the rank convention of the p-quantile, the clamp constants of the
// base, the 3-bit layout, the +1/-1 orientation of the signed DE codebook.
//
// Build: g++ -O2 -std=c++17 -ffp-contract=off -fPIC -shared -pthread

#include <algorithm>
#include <cmath>
#include <cstdint>
#include <cstring>
#include <thread>
#include <vector>

namespace {

inline uint32_t f2u(float x) { uint32_t u; std::memcpy(&u, &x, 4); return u; }
inline float u2f(uint32_t u) { float x; std::memcpy(&x, &u, 4); return x; }

// ---------------------------------------------------------------------------
// Codebooks (Appendix A).
// ---------------------------------------------------------------------------
enum Codebook {
    CB_DE_SIGNED = 0,      // signed dynamic exponent: first moment (Sec. 3.4)
    CB_DE_UNSIGNED = 1,    // unsigned dynamic exponent (baseline)
    CB_LINEAR_UNSIGNED = 2,// {0, 1/(2^b-1), ..., 1}
    CB_LINEAR_SIGNED = 3,  // {0, +-1/(2^(b-1)-1), ..., +-1}
    CB_LINEAR_NOZERO = 4   // {1/2^b, ..., 1} (the 4-bit Adam variant)
};

// One positive dynamic-exponent magnitude (Appendix A, "Dynamic exponent
// mapping"): E leading zero bits give the decade 10^-E; the F fraction bits
// index 2^F equal cells of [0.1, 1] and the level is the cell's midpoint.
//   value = (0.1 + (j + 1/2) * 0.9 / 2^F) / 10^E
//         = (2^(F+1) + 9 (2j+1)) / (10^(E+1) * 2^(F+1))      (exact rational)
// evaluated as one binary64 division of two exact integers, then rounded to
// binary32.
float de_magnitude(int E, int F, int j) {
    double num = std::ldexp(1.0, F + 1) + 9.0 * (2 * j + 1);
    double den = std::pow(10.0, E + 1) * std::ldexp(1.0, F + 1);
    return (float)(num / den);
}

// Fills levels[0 .. 2^bits) in ascending order; returns the count or -1.
int build_codebook(int kind, int bits, float* levels) {
    if (bits < 1 || bits > 8) return -1;
    const int K = 1 << bits;
    std::vector<float> v;
    if (kind == CB_DE_SIGNED) {
        // One bit is the sign; the remaining bits-1 bits split as E + 1 + F.
        // All-zero magnitude bits give 0; the pattern left over by the sign
        // of zero is used for +1 (the codebook has +1 but not -1).
        if (bits < 2) return -1;
        v.push_back(0.0f);
        v.push_back(1.0f);
        for (int E = 0; E <= bits - 2; ++E) {
            int F = bits - 2 - E;
            for (int j = 0; j < (1 << F); ++j) {
                float a = de_magnitude(E, F, j);
                v.push_back(a);
                v.push_back(-a);
            }
        }
    } else if (kind == CB_DE_UNSIGNED) {
        v.push_back(0.0f);
        v.push_back(1.0f);
        // no sign bit: E + 1 + F = bits with F >= 1; the two patterns not used by a
        // magnitude are 0 and 1
        for (int E = 0; E <= bits - 2; ++E) {
            int F = bits - 1 - E;
            for (int j = 0; j < (1 << F); ++j) v.push_back(de_magnitude(E, F, j));
        }
    } else if (kind == CB_LINEAR_UNSIGNED) {
        for (int k = 0; k < K; ++k) v.push_back((float)((double)k / (double)(K - 1)));
    } else if (kind == CB_LINEAR_SIGNED) {
        // {0, +-1/(2^(b-1)-1), ..., +-1}: 2^b - 1 distinct levels.
        if (bits < 2) return -1;
        int h = (1 << (bits - 1)) - 1;
        for (int k = -h; k <= h; ++k) v.push_back((float)((double)k / (double)h));
    } else if (kind == CB_LINEAR_NOZERO) {
        for (int k = 1; k <= K; ++k) v.push_back((float)((double)k / (double)K));
    } else {
        return -1;
    }
    std::sort(v.begin(), v.end());
    for (size_t i = 0; i < v.size(); ++i) levels[i] = v[i];
    return (int)v.size();
}

// ---------------------------------------------------------------------------
// Base-2 logarithm and exponential in binary32, as fixed operation sequences.
// The kernel rounds log_alpha(x/Delta) + xi to an integer (Eq. 6); for the CPU
// and the GPU to take that decision identically the logarithm must be the same
// function on both sides, so it is specified as IEEE operations only.
// ---------------------------------------------------------------------------

// log2(x) for normal x > 0.  x = 2^e * m with m in [sqrt(1/2), sqrt(2));
// log2(m) = f * P(f), f = m - 1, P of degree 8 evaluated by Horner with fma.
// A NaN is returned as it is (the bit operations below would turn it into a
// number that depends on its sign and payload): in Eq. 6 the clamp then takes the
// unordered value to code 0, whatever produced the NaN.
float log2_sp(float x) {
    if (x != x) return x;
    static const float c[9] = {
        0x1.715476p+0f, -0x1.71547p-1f, 0x1.ec73d6p-2f, -0x1.715c4ep-2f, 0x1.26d384p-2f,
        -0x1.e95be6p-3f, 0x1.b9c91ap-3f, -0x1.a87d0ep-3f, 0x1.01b6dep-3f};
    int32_t i = (int32_t)f2u(x);
    int32_t e = (i - 0x3F3504F3) >> 23;          // arithmetic shift
    float m = u2f((uint32_t)(i - e * 0x00800000));
    float f = m - 1.0f;
    float p = c[8];
    for (int k = 7; k >= 0; --k) p = std::fmaf(p, f, c[k]);
    return std::fmaf(f, p, (float)e);
}

// 2^x for |x| < 120.  n = rint(x), f = x - n in [-1/2, 1/2], 2^f by a degree-6
// polynomial (Horner, fma), then the exponent field is advanced by n.
float exp2_sp(float x) {
    static const float c[7] = {
        0x1p+0f, 0x1.62e43p-1f, 0x1.ebfbdap-3f, 0x1.c6aed4p-5f,
        0x1.3b2dbcp-7f, 0x1.5f456ap-10f, 0x1.41d33cp-13f};
    float n = std::nearbyintf(x);                // round-half-even
    float f = x - n;
    float p = c[6];
    for (int k = 5; k >= 0; --k) p = std::fmaf(p, f, c[k]);
    return u2f(f2u(p) + ((uint32_t)(int32_t)n << 23));
}

// ---------------------------------------------------------------------------
// Philox4x32-10 (Salmon, Moraes, Dror, Shaw: "Parallel random numbers: as easy
// as 1, 2, 3", SC'11).  Counter-based, so any element's draw can be recomputed.
// ---------------------------------------------------------------------------
void philox4x32_10(const uint32_t ctr[4], const uint32_t key[2], uint32_t out[4]) {
    uint32_t c0 = ctr[0], c1 = ctr[1], c2 = ctr[2], c3 = ctr[3];
    uint32_t k0 = key[0], k1 = key[1];
    for (int r = 0; r < 10; ++r) {
        uint64_t p0 = (uint64_t)0xD2511F53u * c0;
        uint64_t p1 = (uint64_t)0xCD9E8D57u * c2;
        uint32_t n0 = (uint32_t)(p1 >> 32) ^ c1 ^ k0;
        uint32_t n1 = (uint32_t)p1;
        uint32_t n2 = (uint32_t)(p0 >> 32) ^ c3 ^ k1;
        uint32_t n3 = (uint32_t)p0;
        c0 = n0; c1 = n1; c2 = n2; c3 = n3;
        k0 += 0x9E3779B9u;
        k1 += 0xBB67AE85u;
    }
    out[0] = c0; out[1] = c1; out[2] = c2; out[3] = c3;
}

enum Purpose { PURPOSE_V = 0, PURPOSE_M = 1, PURPOSE_P = 2 };

// The 16-bit draw that belongs to element `idx` of tensor `tensor` at `step`.
// One Philox call serves eight consecutive elements:
// key = seed, counter = (idx/8 low, idx/8 high, step, 4*tensor + purpose);
// element idx takes halfword idx mod 8 of the 128 output bits, i.e. the low
// (even idx) or high (odd idx) half of output word (idx mod 8) / 2.
uint32_t philox_draw16(uint64_t seed, int64_t step, int32_t tensor, int64_t idx, int purpose) {
    uint64_t q = (uint64_t)idx >> 3;
    uint32_t ctr[4] = {(uint32_t)q, (uint32_t)(q >> 32), (uint32_t)step,
                       (uint32_t)tensor * 4u + (uint32_t)purpose};
    uint32_t key[2] = {(uint32_t)seed, (uint32_t)(seed >> 32)};
    uint32_t out[4];
    philox4x32_10(ctr, key, out);
    uint32_t w = out[(idx & 7) >> 1];
    return (idx & 1) ? (w >> 16) : (w & 0xFFFFu);
}

// xi ~ U(-1/2, 1/2) of Eq. 6 from a 16-bit draw d: the midpoints of 2^16 equal
// cells of [-1/2, 1/2], a symmetric grid that never touches +-1/2.  Every value
// is exact in binary32.
inline float xi_from_draw(uint32_t d) {
    return (float)(d & 0xFFFFu) * 0x1p-16f - 0.5f + 0x1p-17f;
}
// u ~ U[0, 1) for Eq. 5 from a 16-bit draw.
inline float u_from_draw(uint32_t d) { return (float)(d & 0xFFFFu) * 0x1p-16f; }

// ---------------------------------------------------------------------------
// Quantizers.
// ---------------------------------------------------------------------------

// Eq. 1: index of the level nearest to r, levels ascending.  Written as the
// number of midpoints below r, which is the first argmin (ties go to the lower
// index).
int quant_nearest(const float* y, int K, float r) {
    int q = 0;
    for (int k = 0; k + 1 < K; ++k) {
        float mid = 0.5f * (y[k] + y[k + 1]);
        if (r > mid) ++q;
    }
    return q;
}

// Eq. 5: stochastic rounding between the two levels that bracket r; u in [0,1).
// Outside the codebook's range r is clamped to the end level.
int quant_stochastic(const float* y, int K, float r, float u) {
    int j = 0;
    for (int k = 1; k + 1 < K; ++k)
        if (r >= y[k]) j = k;                    // y[j] <= r < y[j+1], 0 <= j <= K-2
    float inv_gap = 1.0f / (y[j + 1] - y[j]);
    float frac = (r - y[j]) * inv_gap;
    return j + (u < frac ? 1 : 0);
}

// alpha^q by square-and-multiply over the bits of q, least significant first.
float pow_sm(float alpha, int q) {
    float result = 1.0f, base = alpha;
    while (q) {
        if (q & 1) result = result * base;
        base = base * base;
        q >>= 1;
    }
    return result;
}

const float TINY = 0x1p-100f;                    // below this a scale counts as zero
const float RHO_MIN = 0x1p-48f;                  // clamp of x_p / Delta (base > 0)
const float RHO_MAX = 1.0f - 0x1p-10f;           // clamp of x_p / Delta (base < 1)

// Eq. 6, second line: Clip(round_half_even(log_alpha(r) + xi); 0, K-1), with
// log_alpha(r) = log2(r) * (1 / log2(alpha)).  r below 2^-100 (a zero among
// non-zeros) takes the smallest level, K-1: the codebook alpha^k has no zero.
int quant_log(float r, float inv_lambda, float xi, int K) {
    if (r < TINY) return K - 1;
    float t = std::fmaf(log2_sp(r), inv_lambda, xi);
    t = std::fmin(std::fmax(t, 0.0f), (float)(K - 1));
    return (int)std::nearbyintf(t);
}

// Base of the logarithmic codebook from the p-quantile (Sec. 3.2.2):
// alpha = (x_p / Delta)^(1 / (2^b - 1)), so that level K-1 sits on the quantile.
// Returns alpha and, through inv_lambda, 1 / log2(alpha) of the STORED alpha.
float log_base(float x_p, float inv_delta, int K, float* inv_lambda) {
    float rho = x_p * inv_delta;
    rho = std::fmin(std::fmax(rho, RHO_MIN), RHO_MAX);
    float lam = log2_sp(rho) * (1.0f / (float)(K - 1));
    float alpha = exp2_sp(lam);
    *inv_lambda = 1.0f / log2_sp(alpha);
    return alpha;
}

// ---------------------------------------------------------------------------
// Packed codes: element e of a block occupies bits [e*b, e*b + b) of the
// block's little-endian bit string (B*b/8 bytes per block).
// ---------------------------------------------------------------------------
int get_code(const uint8_t* blk, int e, int b) {
    int bit = e * b, v = 0;
    for (int i = 0; i < b; ++i, ++bit) v |= ((blk[bit >> 3] >> (bit & 7)) & 1) << i;
    return v;
}
void set_code(uint8_t* blk, int e, int b, int v) {
    int bit = e * b;
    for (int i = 0; i < b; ++i, ++bit) {
        blk[bit >> 3] = (uint8_t)(blk[bit >> 3] & ~(1u << (bit & 7)));
        blk[bit >> 3] = (uint8_t)(blk[bit >> 3] | (((v >> i) & 1u) << (bit & 7)));
    }
}

inline float bf16_to_float(uint16_t h) { return u2f((uint32_t)h << 16); }
inline uint16_t float_to_bf16(float x) {         // round to nearest, ties to even
    uint32_t u = f2u(x);
    if ((u & 0x7FFFFFFFu) > 0x7F800000u) return (uint16_t)((u >> 16) | 0x0040u);
    return (uint16_t)((u + 0x7FFFu + ((u >> 16) & 1u)) >> 16);
}

// Stochastic rounding of a binary32 value to bf16 with a 16-bit draw d: the two
// neighbouring bf16 values are the truncation and the next pattern away from
// zero; the upper one is taken with probability (dropped 16 bits) / 2^16, so the
// expectation over d is the value itself.  Adding d to the pattern and
// truncating does exactly that (the carry reaches bit 16 iff d >= 2^16 - low
// bits).  A value already representable is returned unchanged; the largest
// finite magnitudes can round to infinity; infinities and NaN are truncated
// (NaN kept quiet).  Not from the paper: its 16-bit baseline is plain BF16
// (Sec. 4, "Baselines"); this is the usual companion of bf16 parameters without
// a binary32 master copy.
inline uint16_t float_to_bf16_sr(float x, uint32_t d) {
    uint32_t u = f2u(x);
    if ((u & 0x7F800000u) == 0x7F800000u)
        return (uint16_t)((u >> 16) | ((u & 0x007FFFFFu) ? 0x0040u : 0u));
    return (uint16_t)((u + (d & 0xFFFFu)) >> 16);
}

// max over the block of the bit patterns of |x|: equal to the numerical maximum
// for finite values, and a NaN if any element is NaN.
inline float absmax_bits(const float* x, int n) {
    uint32_t m = 0;
    for (int i = 0; i < n; ++i) m = std::max(m, f2u(x[i]) & 0x7FFFFFFFu);
    return u2f(m);
}

// Second-moment codebook selector of the hyper-parameter record -> Codebook, or
// -1 for the logarithmic quantizer.
inline int v_codebook_kind(int sel) {
    return sel == 1 ? CB_DE_UNSIGNED : sel == 2 ? CB_LINEAR_UNSIGNED : sel == 3 ? CB_LINEAR_NOZERO : -1;
}

}  // namespace

extern "C" {

uint32_t so_bf16_sr(float x, uint32_t d) { return float_to_bf16_sr(x, d); }
uint32_t so_bf16_rn(float x) { return float_to_bf16(x); }

// Mirrors the hyper-parameter record of the library's C ABI (declared here
// independently; the two must agree field by field).
struct so_hyper {
    float lr, beta1, beta2, eps, weight_decay;
    float p_quantile;
    float fixed_alpha;    // in (0,1): keep this base for every block (no quantile); otherwise 0
    int32_t adamw, bias_correction, round_m, round_v, param_dtype;
    int32_t belief;       // 0: Adam(W); 1: AdaBelief (second moment tracks (g - m^)^2 + eps)
    int32_t param_round;  // bf16 parameters: 0 round to nearest even, 1 stochastic (Philox purpose 2)
    int32_t v_codebook;   // second moment: 0 logarithmic, Eq. 6 (SOLO); 1 unsigned DE, 2 linear,
                          // 3 linear without zero -- the baselines of Sec. 4, nearest rounding (Eq. 1)
    uint64_t seed;
};

int so_codebook(int kind, int bits, float* levels) { return build_codebook(kind, bits, levels); }
float so_log2_sp(float x) { return log2_sp(x); }
float so_exp2_sp(float x) { return exp2_sp(x); }
void so_philox4x32_10(const uint32_t* ctr, const uint32_t* key, uint32_t* out) {
    philox4x32_10(ctr, key, out);
}
uint32_t so_philox_draw16(uint64_t seed, int64_t step, int32_t tensor, int64_t idx, int purpose) {
    return philox_draw16(seed, step, tensor, idx, purpose);
}
float so_xi(uint32_t d) { return xi_from_draw(d); }
float so_u(uint32_t d) { return u_from_draw(d); }
int so_quant_nearest(const float* y, int K, float r) { return quant_nearest(y, K, r); }
int so_quant_stochastic(const float* y, int K, float r, float u) {
    return quant_stochastic(y, K, r, u);
}
int so_quant_log(float r, float inv_lambda, float xi, int K) {
    return quant_log(r, inv_lambda, xi, K);
}
float so_pow_sm(float alpha, int q) { return pow_sm(alpha, q); }
float so_log_base(float x_p, float delta, int K, float* inv_lambda) {
    return log_base(x_p, 1.0f / delta, K, inv_lambda);
}
int so_get_code(const uint8_t* blk, int e, int b) { return get_code(blk, e, b); }
void so_set_code(uint8_t* blk, int e, int b, int v) { set_code(blk, e, b, v); }

// Bytes of optimizer state for `numel` elements: packed codes of both moments
// (a full slot for every block, tail included) plus three binary32 words per
// block (Delta_m, Delta_v, alpha).  Sec. 4.2 "Block size": one binary32 scale
// costs 1/4 bit per element at block 128, SOLO's buffered base doubles that
// for the second moment.
int so_state_bytes(int64_t numel, int bits_m, int bits_v, int block, uint64_t* out) {
    if (numel < 0 || block <= 0) return -1;
    int64_t nblk = (numel + block - 1) / block;
    *out = (uint64_t)nblk * (uint64_t)(block * bits_m / 8) +
           (uint64_t)nblk * (uint64_t)(block * bits_v / 8) + 12u * (uint64_t)nblk;
    return 0;
}

// Eq. 7: the largest beta' with beta'/(1-beta') r_med(b') <= beta/(1-beta) r_med(b).
double so_beta_prime(double beta, double r_med_b, double r_med_bprime) {
    double c = beta / (1.0 - beta) * r_med_b / r_med_bprime;
    return c / (1.0 + c);
}

// ---------------------------------------------------------------------------
// The optimizer step on a slice of one tensor (Sec. 3.1 Eq. 2-4, Sec. 3.4).
//
// The slice holds elements [elem_offset, elem_offset + n) of tensor number
// `tensor`; elem_offset is a multiple of `block`, so the slice starts on a block
// boundary and only its last block can be short.  codes_*/scale_*/alpha point at
// the slice's first block.  Blocks [blk_lo, blk_hi) of the slice are processed
// (so that threads can split the work); everything else is left untouched.
//
// Per block, in this order:
//   dequantize m, v  (Eq. 2)           m~ = y[q_m] Delta_m,  v~ = alpha^q_v Delta_v
//   EMA              (Eq. 3)           m^ = b1 m~ + (1-b1) g,  v^ = b2 v~ + (1-b2) g^2
//   Adam(W) update with m^, v^         p <- p (1 - lr wd) - (lr/bc1) m^ / (sqrt(v^)/sqrt(bc2) + eps)
//   new scales                          Delta_m' = max |m^|,  Delta_v' = max v^
//   new base from the p-quantile        alpha' = (x_p / Delta_v')^(1/(K_v - 1))
//   quantize         (Eq. 4)           m: Eq. 1 (or Eq. 5),  v: Eq. 6
// Optional outputs (may be null): m_hat, v_hat (n floats each), and flags (n
// bytes; bit 0 / bit 1 set when the m / v value lies within 1e-6 relative of a
// rounding boundary, evaluated in binary64).
// Full-precision switch: when m32 and v32 are given (n floats each) the moments
// are read from and written to them unquantized and the packed state is ignored;
// the EMA and the parameter update are the same lines of code, so this mode is
// what ties them to a textbook Adam(W).
// ---------------------------------------------------------------------------
static void step_blocks(void* param, const uint16_t* grad, int64_t n, int64_t elem_offset,
                        int32_t tensor, int bits_m, int bits_v, int block, uint8_t* codes_m,
                        uint8_t* codes_v, float* scale_m, float* scale_v, float* alpha,
                        const so_hyper* h, int64_t step, int64_t blk_lo, int64_t blk_hi,
                        float* m_hat_out, float* v_hat_out, uint8_t* flags, float* m32,
                        float* v32) {
    const int Km = 1 << bits_m, Kv = 1 << bits_v;
    float ym[256], yv[256];
    build_codebook(CB_DE_SIGNED, bits_m, ym);
    const int v_kind = v_codebook_kind(h->v_codebook);          // < 0: logarithmic (SOLO)
    if (v_kind >= 0) build_codebook(v_kind, bits_v, yv);

    // Hyper-parameter scalars: binary64, rounded once.
    const double t = (double)step;
    const double bc1 = h->bias_correction ? 1.0 - std::pow((double)h->beta1, t) : 1.0;
    const double bc2 = h->bias_correction ? 1.0 - std::pow((double)h->beta2, t) : 1.0;
    const float step_size = (float)((double)h->lr / bc1);
    const float inv_sqrt_bc2 = (float)(1.0 / std::sqrt(bc2));
    const float decay = h->adamw ? (float)(1.0 - (double)h->lr * (double)h->weight_decay) : 1.0f;
    const float b1 = h->beta1, b2 = h->beta2;
    const float omb1 = 1.0f - b1, omb2 = 1.0f - b2;
    const bool l2 = !h->adamw && h->weight_decay != 0.0f;

    const size_t slot_m = (size_t)block * bits_m / 8, slot_v = (size_t)block * bits_v / 8;
    std::vector<float> mh(block), vh(block), sorted(block);

    for (int64_t j = blk_lo; j < blk_hi; ++j) {
        const int64_t e0 = j * block;
        const int nb = (int)std::min<int64_t>(block, n - e0);
        uint8_t* cm = codes_m + (size_t)j * slot_m;
        uint8_t* cv = codes_v + (size_t)j * slot_v;
        const float dm = scale_m[j], dv = scale_v[j], al = alpha[j];

        for (int e = 0; e < nb; ++e) {
            const int64_t i = e0 + e;
            float p = h->param_dtype == 1 ? bf16_to_float(((uint16_t*)param)[i])
                                          : ((float*)param)[i];
            float g = bf16_to_float(grad[i]);
            if (l2) g = std::fmaf(h->weight_decay, p, g);       // Adam: L2 term in the gradient
            // Eq. 2 (or, with the full-precision switch, the stored binary32 moments)
            float m_t = m32 ? m32[i] : ym[get_code(cm, e, bits_m)] * dm;
            float v_t = v32 ? v32[i]
                      : v_kind >= 0 ? yv[get_code(cv, e, bits_v)] * dv
                                    : pow_sm(al, get_code(cv, e, bits_v)) * dv;
            // Eq. 3.  AdaBelief (Sec. 4.2, "AdaBelief"; Zhuang et al. 2020): the unsigned EMA's
            // signal is (g - m^)^2 instead of g^2 and eps is added to the state at every step
            float m_h = std::fmaf(b1, m_t, omb1 * g);
            float sig = h->belief ? g - m_h : g;
            float v_h = std::fmaf(b2, v_t, omb2 * (sig * sig));
            if (h->belief) v_h = v_h + h->eps;
            mh[e] = m_h;
            vh[e] = v_h;
            // Adam(W) with the un-requantized moments
            float den = std::fmaf(std::sqrt(v_h), inv_sqrt_bc2, h->eps);
            float p_new = std::fmaf(-step_size, m_h / den, p * decay);
            if (h->param_dtype == 1) {
                ((uint16_t*)param)[i] =
                    h->param_round
                        ? float_to_bf16_sr(p_new, philox_draw16(h->seed, step, tensor,
                                                                elem_offset + i, PURPOSE_P))
                        : float_to_bf16(p_new);
            } else {
                ((float*)param)[i] = p_new;
            }
        }
        if (m_hat_out) std::copy(mh.begin(), mh.begin() + nb, m_hat_out + e0);
        if (v_hat_out) std::copy(vh.begin(), vh.begin() + nb, v_hat_out + e0);
        if (flags) std::fill(flags + e0, flags + e0 + nb, (uint8_t)0);
        if (m32) {                                               // no quantization at all
            std::copy(mh.begin(), mh.begin() + nb, m32 + e0);
            std::copy(vh.begin(), vh.begin() + nb, v32 + e0);
            continue;
        }

        std::memset(cm, 0, slot_m);
        std::memset(cv, 0, slot_v);

        // ---- first moment: Delta = max |m^| (Sec. 3.1), Eq. 1 or Eq. 5 ----
        float dm_new = absmax_bits(mh.data(), nb);
        if (dm_new < TINY) {
            scale_m[j] = 0.0f;                                   // vanishing block: all codes 0
        } else {
            scale_m[j] = dm_new;
            const float inv = 1.0f / dm_new;
            for (int e = 0; e < nb; ++e) {
                float r = mh[e] * inv;
                int q;
                if (h->round_m) {
                    uint32_t d = philox_draw16(h->seed, step, tensor, elem_offset + e0 + e, PURPOSE_M);
                    q = quant_stochastic(ym, Km, r, u_from_draw(d));
                } else {
                    q = quant_nearest(ym, Km, r);
                    if (flags) {
                        for (int k = 0; k + 1 < Km; ++k) {
                            double mid = 0.5 * ((double)ym[k] + (double)ym[k + 1]);
                            if (std::fabs((double)r - mid) <= 1e-6 * std::fabs(mid)) flags[e0 + e] |= 1;
                        }
                    }
                }
                set_code(cm, e, bits_m, q);
            }
        }

        // ---- second moment: Delta = max v^, base from the p-quantile, Eq. 6 ----
        float dv_new = absmax_bits(vh.data(), nb);
        if (dv_new < TINY) {
            scale_v[j] = 0.0f;
            alpha[j] = 0.5f;
        } else if (v_kind >= 0) {
            // baseline: block-wise absmax scaling and the nearest level of a fixed codebook
            // (Eq. 1; Sec. 4, "Baselines"); the base is not used and keeps its initial value
            scale_v[j] = dv_new;
            alpha[j] = 0.5f;
            const float inv = 1.0f / dv_new;
            for (int e = 0; e < nb; ++e) {
                float r = vh[e] * inv;
                set_code(cv, e, bits_v, quant_nearest(yv, Kv, r));
                if (flags) {
                    for (int k = 0; k + 1 < Kv; ++k) {
                        double mid = 0.5 * ((double)yv[k] + (double)yv[k + 1]);
                        if (std::fabs((double)r - mid) <= 1e-6 * std::fabs(mid)) flags[e0 + e] |= 2;
                    }
                }
            }
        } else {
            scale_v[j] = dv_new;
            const float inv = 1.0f / dv_new;
            float inv_lambda, al_new;
            if (h->fixed_alpha > 0.0f && h->fixed_alpha < 1.0f) {
                // standard logarithmic quantization with a fixed base (Sec. 3.2.2, the remark on
                // alpha = 1/2; the setting of Prop. 3.5)
                al_new = h->fixed_alpha;
                inv_lambda = 1.0f / log2_sp(al_new);
            } else {
                // p-quantile as an order statistic: the k-th smallest, k = max(1, ceil(p n)).
                int64_t k = (int64_t)std::ceil((double)h->p_quantile * (double)nb);
                k = std::min<int64_t>(std::max<int64_t>(k, 1), nb);
                std::copy(vh.begin(), vh.begin() + nb, sorted.begin());
                std::sort(sorted.begin(), sorted.begin() + nb,
                          [](float a, float b) { return f2u(a) < f2u(b); });
                float x_p = sorted[k - 1];
                al_new = log_base(x_p, inv, Kv, &inv_lambda);
            }
            alpha[j] = al_new;
            for (int e = 0; e < nb; ++e) {
                float r = vh[e] * inv;
                float xi = 0.0f;
                if (h->round_v) {
                    uint32_t d = philox_draw16(h->seed, step, tensor, elem_offset + e0 + e, PURPOSE_V);
                    xi = xi_from_draw(d);
                }
                int q = quant_log(r, inv_lambda, xi, Kv);
                set_code(cv, e, bits_v, q);
                if (flags && !(r < TINY)) {
                    // distance of t to the nearest half-integer, in units of relative change of r
                    double tt = std::log2((double)r) * (double)inv_lambda + (double)xi;
                    double frac = std::fabs(tt - std::floor(tt) - 0.5);
                    if (tt > -0.5 && tt < (double)Kv - 0.5 &&
                        frac * std::fabs(1.0 / (double)inv_lambda) * 0.6931471805599453 <= 1e-6)
                        flags[e0 + e] |= 2;
                }
            }
        }
    }
}

int so_step(void* param, const uint16_t* grad, int64_t n, int64_t elem_offset, int32_t tensor,
            int bits_m, int bits_v, int block, uint8_t* codes_m, uint8_t* codes_v, float* scale_m,
            float* scale_v, float* alpha, const so_hyper* h, int64_t step, int nthreads,
            float* m_hat_out, float* v_hat_out, uint8_t* flags, float* m32, float* v32) {
    if ((m32 == nullptr) != (v32 == nullptr)) return -1;
    if (n < 0 || block <= 0 || (block * bits_m) % 8 || (block * bits_v) % 8) return -1;
    if (bits_m < 2 || bits_m > 8 || bits_v < 1 || bits_v > 8 || elem_offset % block) return -1;
    if (h->v_codebook < 0 || h->v_codebook > 3) return -1;
    const int64_t nblk = (n + block - 1) / block;
    if (nthreads <= 1 || nblk < 2) {
        step_blocks(param, grad, n, elem_offset, tensor, bits_m, bits_v, block, codes_m, codes_v,
                    scale_m, scale_v, alpha, h, step, 0, nblk, m_hat_out, v_hat_out, flags, m32, v32);
        return 0;
    }
    // Blocks are independent: contiguous ranges of blocks, one plain thread each.
    std::vector<std::thread> pool;
    const int64_t per = (nblk + nthreads - 1) / nthreads;
    for (int t = 0; t < nthreads; ++t) {
        int64_t lo = t * per, hi = std::min<int64_t>(nblk, lo + per);
        if (lo >= hi) break;
        pool.emplace_back(step_blocks, param, grad, n, elem_offset, tensor, bits_m, bits_v, block,
                          codes_m, codes_v, scale_m, scale_v, alpha, h, step, lo, hi, m_hat_out,
                          v_hat_out, flags, m32, v32);
    }
    for (auto& th : pool) th.join();
    return 0;
}

// Eq. 2 for inspection: which = 0 first moment, 1 second moment.
// v_codebook: the selector the second moment was written with (0 = logarithmic).
int so_dequant(int which, int64_t n, int bits, int block, const uint8_t* codes, const float* scale,
               const float* alpha, int v_codebook, float* out) {
    float ym[256];
    if (which == 0 && build_codebook(CB_DE_SIGNED, bits, ym) < 0) return -1;
    const int v_kind = v_codebook_kind(v_codebook);
    if (which == 1 && v_kind >= 0) {
        if (build_codebook(v_kind, bits, ym) < 0) return -1;
        which = 0;                                               // table lookup from here on
    }
    const size_t slot = (size_t)block * bits / 8;
    for (int64_t i = 0; i < n; ++i) {
        int64_t j = i / block;
        int q = get_code(codes + (size_t)j * slot, (int)(i % block), bits);
        out[i] = which == 0 ? ym[q] * scale[j] : pow_sm(alpha[j], q) * scale[j];
    }
    return 0;
}

int so_hardware_threads(void) { return (int)std::thread::hardware_concurrency(); }

// ---------------------------------------------------------------------------
// Generic quantized EMA on ONE quantization unit of any length (Eq. 2-4 with a
// chosen codebook).  Used only by the tests that reproduce the paper's analysis:
// signal swamping (Thm 3.1, Cor. 3.2, Example 3.3), exact decay (Prop. 3.5) and
// stochastic rounding (Thm 3.6).
//   mode 0: nearest rounding (Eq. 1) on codebook `kind`
//   mode 1: stochastic rounding (Eq. 5) on codebook `kind`, u from the upper
//           halves of `rnd` (n words, one 16-bit draw each)
//   mode 2: SOLO logarithmic quantizer (Eq. 6), xi from `rnd` likewise (null: xi = 0);
//           fixed_alpha > 0 keeps that base, otherwise the base comes from the
//           p-quantile of the new values.
// codes: one int per element (unpacked).  delta/alpha: in/out scalars.
// ---------------------------------------------------------------------------
int so_qema(int mode, int kind, int bits, int64_t n, int32_t* codes, float* delta, float* alpha,
            const float* z, float beta, float p_quantile, float fixed_alpha, const uint32_t* rnd,
            float* x_hat_out) {
    const int K0 = 1 << bits;
    float y[256];
    int K = K0;
    if (mode != 2) {
        K = build_codebook(kind, bits, y);
        if (K < 0) return -1;
    }
    std::vector<float> xh((size_t)n);
    const float omb = 1.0f - beta;
    for (int64_t i = 0; i < n; ++i) {
        float x_t = mode == 2 ? pow_sm(*alpha, codes[i]) * *delta : y[codes[i]] * *delta;
        xh[i] = std::fmaf(beta, x_t, omb * z[i]);
    }
    if (x_hat_out) std::copy(xh.begin(), xh.end(), x_hat_out);
    float d = absmax_bits(xh.data(), (int)n);
    if (d < TINY) {
        *delta = 0.0f;
        if (mode == 2 && !(fixed_alpha > 0.0f)) *alpha = 0.5f;
        for (int64_t i = 0; i < n; ++i) codes[i] = 0;
        return 0;
    }
    *delta = d;
    const float inv = 1.0f / d;
    if (mode == 2) {
        float inv_lambda;
        if (fixed_alpha > 0.0f) {
            *alpha = fixed_alpha;
            inv_lambda = 1.0f / log2_sp(fixed_alpha);
        } else {
            int64_t k = (int64_t)std::ceil((double)p_quantile * (double)n);
            k = std::min<int64_t>(std::max<int64_t>(k, 1), n);
            std::vector<float> s(xh);
            std::sort(s.begin(), s.end(), [](float a, float b) { return f2u(a) < f2u(b); });
            *alpha = log_base(s[k - 1], inv, K0, &inv_lambda);
        }
        for (int64_t i = 0; i < n; ++i)
            codes[i] = quant_log(xh[i] * inv, inv_lambda, rnd ? xi_from_draw(rnd[i] >> 16) : 0.0f, K0);
    } else {
        for (int64_t i = 0; i < n; ++i) {
            float r = xh[i] * inv;
            codes[i] = mode == 1 ? quant_stochastic(y, K, r, u_from_draw(rnd[i] >> 16))
                                 : quant_nearest(y, K, r);
        }
    }
    return 0;
}

}  // extern "C"
