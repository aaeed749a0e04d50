// CPU oracle for the BF16 + stochastic-rounding AdamW update.
//
// THIS FILE IS TEST INFRASTRUCTURE, NOT THE PRODUCT.  It is a plain, slow, one-element-at-a-time
// restatement of what the update computes, written from the paper's definitions so that a reader
// can check it by eye.  It shares no code, header, table or helper with the CUDA library and the
// CUDA library never calls it.  Only the test-suite, the smoke check and the benchmark's
// CPU-baseline leg load it.
//
// What is defined here, and the passage each item follows:
//   oracle_philox4x32_10      Philox4x32 with 10 rounds (Salmon, Moraes, Dror, Shaw, SC'11).  All
//                             Algorithm 1 requires (its REQUIRE list and the r <- r^(opt) step) is
//                             an optimizer random state that every replica holds identically; a
//                             counter-based generator gives that by construction.
//   oracle_sr_bf16_bits       stochastic rounding Q_SR of Eq. 2, realised the way Section 3
//                             describes it: take the FP32 value, add uniform noise below the bits
//                             that BF16 keeps, shift the fraction out.
//   oracle_rne_bf16_bits      nearest rounding Q of Eq. 1 in its IEEE round-half-to-even form.
//   oracle_adamw_scalars      the per-iteration scalars of Algorithm 1 (bias corrections of the
//                             m-hat and v-hat steps, alpha_t * lambda).
//   oracle_adamw_element      one element of Algorithm 1 (moment updates, bias-corrected
//                             direction, decoupled decay), in FP32, before any rounding.
//   oracle_adamw_step         Algorithm 1 over an array: element function + Q_SR on x, m and v.
//   oracle_sr_downcast        Q_SR applied to an FP32 array.
//   oracle_sr_downcast_fp8    Q_SR of Eq. 2 on the 8-bit grids E4M3 and E5M2, and
//   oracle_sr_downcast_fp4    on the 4-bit grid E2M1 (the conclusion names FP8/4 as the next targets).
//   oracle_sr_accumulate      Q_SR (or Q) applied to a BF16 accumulator plus a new term (Section 3
//                             keeps the accumulated gradient in BF16 too).
//   oracle_master_adamw_step  the mixed-precision recipe the paper compares against.
//   oracle_sqnorm             sum of squares of the gradient with a fixed summation tree
//   oracle_clip_scale         global-norm clipping coefficient.  (Neither is in the paper; they
//                             are the usual companions of the update and are defined below.)
//
// Floating point: FP32 round-to-nearest-even for the element function (Section 3: the update is
// evaluated in FP32 and only its results are rounded), no flush-to-zero, no contraction except where
// fmaf is written.
// Build with -ffp-contract=off and without -ffast-math.
//
// Pins (tests/, run without a GPU): Philox known-answer vectors of its authors; Eq. 2's two-neighbour
// property, exact P(up), exact mean (unbiasedness) and exact variance by enumerating all 65536
// noise values; the stagnation and random-walk examples of Section 2; every FP32 intermediate of
// the element function against correctly rounded exact rational arithmetic; the step-1 closed
// form; a library AdamW as a loose bound; the summation tree against exact integer arithmetic and,
// for the ORDER of its additions, against a restatement of the rule on order-sensitive data; the
// rounding decisions of elements and slots that share a Philox call for pairwise independence.
// Not pinned by the paper (its Algorithm 1 is ambiguous there; "parity unpinned" for that choice
// alone): where epsilon sits relative to the square root.  The default is the AdamW convention of
// the optimizer the paper cites, sqrt(v/(1-beta2^t)) + epsilon; flag bit 3 selects the other reading,
// sqrt(v/(1-beta2^t) + epsilon), the form of the paper's analysis.  Both are pinned arithmetically
// (exact rational intermediates, closed forms); which one the paper's experiments ran is not.

#include <cmath>
#include <cstdint>
#include <cstring>

#ifdef _OPENMP
#include <omp.h>
#endif

namespace {

inline uint32_t bits_of(float x) {
    uint32_t b;
    std::memcpy(&b, &x, sizeof b);
    return b;
}

inline float float_of(uint32_t b) {
    float x;
    std::memcpy(&x, &b, sizeof x);
    return x;
}

inline float bf16_to_float(uint16_t h) { return float_of(static_cast<uint32_t>(h) << 16); }

inline bool is_nan_bits(uint32_t b) { return (b & 0x7FFFFFFFu) > 0x7F800000u; }

constexpr uint16_t kCanonicalNaN = 0x7FC0;

// ---- Philox4x32-10 -------------------------------------------------------------------------
// One round maps the counter (c0,c1,c2,c3) under the round key (k0,k1) to
//   ( hi(M1*c2) ^ c1 ^ k0,  lo(M1*c2),  hi(M0*c0) ^ c3 ^ k1,  lo(M0*c0) )
// with 32x32->64 bit products; between rounds the key advances by the Weyl constants.
void philox4x32_10(const uint32_t ctr[4], const uint32_t key[2], uint32_t out[4]) {
    const uint64_t M0 = 0xD2511F53u, M1 = 0xCD9E8D57u;
    const uint32_t W0 = 0x9E3779B9u, W1 = 0xBB67AE85u;
    uint32_t c0 = ctr[0], c1 = ctr[1], c2 = ctr[2], c3 = ctr[3];
    uint32_t k0 = key[0], k1 = key[1];
    for (int round = 0; round < 10; ++round) {
        if (round > 0) {
            k0 += W0;
            k1 += W1;
        }
        const uint64_t p0 = M0 * c0;
        const uint64_t p1 = M1 * c2;
        const uint32_t n0 = static_cast<uint32_t>(p1 >> 32) ^ c1 ^ k0;
        const uint32_t n1 = static_cast<uint32_t>(p1);
        const uint32_t n2 = static_cast<uint32_t>(p0 >> 32) ^ c3 ^ k1;
        const uint32_t n3 = static_cast<uint32_t>(p0);
        c0 = n0; c1 = n1; c2 = n2; c3 = n3;
    }
    out[0] = c0; out[1] = c1; out[2] = c2; out[3] = c3;
}

// ---- the optimizer's random state r^(opt)_t ------------------------------------------------
// Algorithm 1 needs a random state that is the same on every replica at iteration t.  Here the
// state is a pure function of (seed, step, tensor_id, global element index).  One Philox call
// yields 128 bits = eight 16-bit noise values, so one call serves one rounding slot (0: x, 1: m,
// 2: v) of a group of eight consecutive elements:
//   group   = index >> 3,   e = index & 7
//   number  = 4 * group + slot                       (a 64-bit integer)
//   key     = (seed[31:0], step)
//   counter = (number[31:0], number[63:32], tensor_id, seed[63:32])
// Elements 2j and 2j+1 of the group share output word j: the even one takes its low 16 bits, the
// odd one its high 16 bits.  Every bit of every call is used exactly once.
uint32_t noise_for_slot(uint64_t seed, uint32_t step, uint32_t tensor_id, uint64_t index, uint32_t slot) {
    const uint64_t group = index >> 3;
    const uint32_t e = static_cast<uint32_t>(index & 7u);
    const uint64_t number = 4u * group + slot;
    const uint32_t ctr[4] = {static_cast<uint32_t>(number), static_cast<uint32_t>(number >> 32),
                             tensor_id, static_cast<uint32_t>(seed >> 32)};
    const uint32_t key[2] = {static_cast<uint32_t>(seed), step};
    uint32_t w[4];
    philox4x32_10(ctr, key, w);
    const uint32_t word = w[e >> 1];
    return (e & 1u) ? (word >> 16) : (word & 0xFFFFu);
}

struct Noise3 { uint32_t rp, rm, rv; };

Noise3 noise_for(uint64_t seed, uint32_t step, uint32_t tensor_id, uint64_t index) {
    return Noise3{noise_for_slot(seed, step, tensor_id, index, 0), noise_for_slot(seed, step, tensor_id, index, 1),
                  noise_for_slot(seed, step, tensor_id, index, 2)};
}

// ---- Eq. 2 by dithering --------------------------------------------------------------------
// BF16 keeps the top 16 bits of the FP32 pattern; the low 16 bits are the position of x between
// its two BF16 neighbours, in units of 2^-16 of their distance.  Adding a uniform integer
// r in [0, 65536) to the pattern carries into the kept bits exactly when low16 + r >= 65536,
// i.e. for low16 of the 65536 values of r: probability (x - floor)/Delta of moving to the
// neighbour away from zero, as Eq. 2 asks.  The pattern is sign-magnitude, so one unsigned add
// serves both signs, crosses binades and the subnormal boundary, and leaves values that are
// already BF16 (low16 == 0), zeros and infinities untouched.  A finite value beyond the largest
// finite BF16 moves to infinity with the same rule.  Any NaN becomes the one quiet NaN 0x7FC0, so
// that the result does not depend on which NaN payload a platform produces.
uint16_t sr_bf16_bits(uint32_t fbits, uint32_t r16) {
    if (is_nan_bits(fbits)) return kCanonicalNaN;
    return static_cast<uint16_t>((fbits + (r16 & 0xFFFFu)) >> 16);
}

// ---- Eq. 1, IEEE form ----------------------------------------------------------------------
// Round to the nearer neighbour; a value exactly half-way goes to the neighbour whose last kept
// bit is zero.
uint16_t rne_bf16_bits(uint32_t fbits) {
    if (is_nan_bits(fbits)) return kCanonicalNaN;
    const uint32_t last_kept = (fbits >> 16) & 1u;
    return static_cast<uint16_t>((fbits + 0x7FFFu + last_kept) >> 16);
}

// beta^t by repeated squaring in double; no libm call, so every platform gets the same bits.
double int_power(double base, uint32_t exponent) {
    double result = 1.0;
    while (exponent != 0) {
        if (exponent & 1u) result *= base;
        base *= base;
        exponent >>= 1;
    }
    return result;
}

}  // namespace

extern "C" {

// Hyper-parameters as the caller states them (Algorithm 1, REQUIRE list; epsilon of the update).
struct oracle_hparams {
    float lr;            // alpha_t
    float beta1;
    float beta2;
    float eps;
    float weight_decay;  // lambda
    uint32_t flags;      // bit0/1/2: stochastic rounding on x / m / v (else nearest-even);
                         // bit3: epsilon under the square root (see oracle_adamw_element)
};

// Scalars that are the same for every element of one iteration.
struct oracle_scalars {
    float beta1;
    float beta2;
    float one_minus_beta1;  // FP32 subtraction
    float one_minus_beta2;
    float step_size;        // alpha_t / (1 - beta1^t)          (the m-hat step folded into alpha_t)
    float rsqrt_bc2;        // 1 / sqrt(1 - beta2^t)            (the v-hat step)
    float eps;
    float lr_wd;            // alpha_t * lambda
    float inv_bc2;          // 1 / (1 - beta2^t)                (the v-hat step without its root)
    uint32_t eps_inside;    // 1: the direction divides by sqrt(v-hat + eps) instead of sqrt(v-hat) + eps
};

// The FP32 intermediates of one element, in the order they are produced.
struct oracle_trace {
    float g;      // gscale * g_in
    float a;      // (1-beta1) * g
    float m_new;  // beta1*m + a                     (moment update for m)
    float b1;     // (1-beta2) * g
    float b2;     // b1 * g
    float v_new;  // beta2*v + b2                    (moment update for v)
    float s;      // sqrt(v_new)                     [epsilon inside: v_new * inv_bc2 + eps]
    float den;    // s * rsqrt_bc2 + eps             [epsilon inside: sqrt(s)]
    float u;      // m_new / den
    float w;      // lr_wd * x
    float q;      // step_size*u + w
    float x_new;  // x - q                           (argument of Q_SR in the update step)
};

int oracle_num_threads(void) {
#ifdef _OPENMP
    return omp_get_max_threads();
#else
    return 1;
#endif
}

void oracle_philox4x32_10(const uint32_t ctr[4], const uint32_t key[2], uint32_t out[4]) {
    philox4x32_10(ctr, key, out);
}

// The three 16-bit noise values (x, m, v) for one element.
void oracle_noise(uint64_t seed, uint32_t step, uint32_t tensor_id, uint64_t index, uint32_t out[3]) {
    const Noise3 r = noise_for(seed, step, tensor_id, index);
    out[0] = r.rp; out[1] = r.rm; out[2] = r.rv;
}

uint32_t oracle_noise_slot(uint64_t seed, uint32_t step, uint32_t tensor_id, uint64_t index, uint32_t slot) {
    return noise_for_slot(seed, step, tensor_id, index, slot);
}

uint16_t oracle_sr_bf16_bits(uint32_t fbits, uint32_t r16) { return sr_bf16_bits(fbits, r16); }

uint16_t oracle_rne_bf16_bits(uint32_t fbits) { return rne_bf16_bits(fbits); }

// Returns 0 on success, 1 for arguments the update is not defined for.
int oracle_adamw_scalars(const oracle_hparams* hp, uint32_t step, oracle_scalars* out) {
    if (step == 0) return 1;  // 1 - beta^0 = 0: the bias correction divides by zero
    const double b1 = hp->beta1, b2 = hp->beta2, lr = hp->lr, wd = hp->weight_decay;
    const double bc1 = 1.0 - int_power(b1, step);
    const double bc2 = 1.0 - int_power(b2, step);
    out->beta1 = hp->beta1;
    out->beta2 = hp->beta2;
    out->one_minus_beta1 = 1.0f - hp->beta1;
    out->one_minus_beta2 = 1.0f - hp->beta2;
    out->step_size = static_cast<float>(lr / bc1);
    out->rsqrt_bc2 = static_cast<float>(1.0 / std::sqrt(bc2));
    out->eps = hp->eps;
    out->lr_wd = static_cast<float>(lr * wd);
    out->inv_bc2 = static_cast<float>(1.0 / bc2);
    out->eps_inside = (hp->flags >> 3) & 1u;
    return 0;
}

// One element of Algorithm 1 in FP32.  Each line is one correctly rounded operation; fmaf is a
// single rounding of a*b+c.
// Where epsilon sits: Algorithm 1 as printed takes a square root in the v-hat step and again divides
// by sqrt(v-hat + eps).  Two readings are implemented.  Default: the AdamW of the optimizer the paper
// cites, sqrt(v/(1-beta2^t)) + eps.  With eps_inside: the form of the paper's analysis (appendix:
// x - alpha_t m / sqrt(eps + v)) with the bias correction of the v-hat step kept,
// sqrt(v/(1-beta2^t) + eps), i.e. the printed update step with the extra root of the v-hat step dropped.
void oracle_adamw_element(float x, float g_in, float m, float v, float gscale,
                          const oracle_scalars* sc, oracle_trace* t) {
    t->g = gscale * g_in;
    t->a = sc->one_minus_beta1 * t->g;
    t->m_new = fmaf(sc->beta1, m, t->a);
    t->b1 = sc->one_minus_beta2 * t->g;
    t->b2 = t->b1 * t->g;
    t->v_new = fmaf(sc->beta2, v, t->b2);
    if (sc->eps_inside) {
        t->s = fmaf(t->v_new, sc->inv_bc2, sc->eps);
        t->den = sqrtf(t->s);
    } else {
        t->s = sqrtf(t->v_new);
        t->den = fmaf(t->s, sc->rsqrt_bc2, sc->eps);
    }
    t->u = t->m_new / t->den;
    t->w = sc->lr_wd * x;
    t->q = fmaf(sc->step_size, t->u, t->w);
    t->x_new = x - t->q;
}

// Algorithm 1 on n elements, in place.  p, m, v hold BF16 bit patterns; g is BF16 (g_is_f32 == 0)
// or FP32 (g_is_f32 == 1).  elem_offset is the global index of element 0, so that a shard of a
// larger buffer draws the same noise as the whole would.
int oracle_adamw_step(uint16_t* p, const void* g, int g_is_f32, uint16_t* m, uint16_t* v, uint64_t n,
                      const oracle_hparams* hp, float gscale, uint64_t seed, uint32_t step,
                      uint32_t tensor_id, uint64_t elem_offset) {
    oracle_scalars sc;
    if (oracle_adamw_scalars(hp, step, &sc) != 0) return 1;
    const uint16_t* g16 = static_cast<const uint16_t*>(g);
    const float* g32 = static_cast<const float*>(g);
    const bool sr_p = hp->flags & 1u, sr_m = hp->flags & 2u, sr_v = hp->flags & 4u;
#pragma omp parallel for schedule(static)
    for (int64_t i = 0; i < static_cast<int64_t>(n); ++i) {
        const float gi = g_is_f32 ? g32[i] : bf16_to_float(g16[i]);
        oracle_trace t;
        oracle_adamw_element(bf16_to_float(p[i]), gi, bf16_to_float(m[i]), bf16_to_float(v[i]), gscale, &sc, &t);
        const Noise3 r = noise_for(seed, step, tensor_id, elem_offset + static_cast<uint64_t>(i));
        p[i] = sr_p ? sr_bf16_bits(bits_of(t.x_new), r.rp) : rne_bf16_bits(bits_of(t.x_new));
        m[i] = sr_m ? sr_bf16_bits(bits_of(t.m_new), r.rm) : rne_bf16_bits(bits_of(t.m_new));
        v[i] = sr_v ? sr_bf16_bits(bits_of(t.v_new), r.rv) : rne_bf16_bits(bits_of(t.v_new));
    }
    return 0;
}

// The mixed-precision comparison recipe the paper measures against (its "O2": FP32 master weights
// and FP32 optimizer states, a BF16 copy of the weights for the forward/backward pass): the same
// element function, results kept in FP32 without any rounding, plus x rounded to nearest (Eq. 1)
// into the BF16 copy.  No random state is involved.
int oracle_master_adamw_step(float* p, uint16_t* p_bf16, const void* g, int g_is_f32, float* m, float* v, uint64_t n,
                             const oracle_hparams* hp, float gscale, uint32_t step) {
    oracle_scalars sc;
    if (oracle_adamw_scalars(hp, step, &sc) != 0) return 1;
    const uint16_t* g16 = static_cast<const uint16_t*>(g);
    const float* g32 = static_cast<const float*>(g);
#pragma omp parallel for schedule(static)
    for (int64_t i = 0; i < static_cast<int64_t>(n); ++i) {
        const float gi = g_is_f32 ? g32[i] : bf16_to_float(g16[i]);
        oracle_trace t;
        oracle_adamw_element(p[i], gi, m[i], v[i], gscale, &sc, &t);
        p[i] = t.x_new;
        m[i] = t.m_new;
        v[i] = t.v_new;
        p_bf16[i] = rne_bf16_bits(bits_of(t.x_new));
    }
    return 0;
}

// ---- Eq. 2 onto an 8-bit floating-point grid -------------------------------------------------
// The paper's closing remark: the method carries over to FP8.  Formats: E4M3 (4 exponent bits,
// bias 7, 3 mantissa bits, no infinity, largest finite 448, S.1111.111 = NaN) and E5M2 (5 exponent
// bits, bias 15, 2 mantissa bits, IEEE-like, largest finite 57344).  For |x| = a with binary
// exponent E, the two neighbouring levels are spaced Delta = 2^(Eq - M), Eq = max(E, 1 - bias)
// (subnormal levels share the spacing of the smallest normal binade).  y = a / Delta = k + f with
// integer k and 0 <= f < 1; Eq. 2 moves to level k + 1 with probability f.  With a uniform 32-bit
// integer r the move happens iff r < floor(f * 2^32), which is exactly probability f whenever f has
// at most 32 fractional bits (every FP32 input down to 2^-12 of the smallest subnormal level) and
// rounds the probability down by less than 2^-32 otherwise.  Magnitudes at or beyond the largest
// finite level saturate to it (E5M2 keeps infinity); NaN gives the pattern 0x7F.
// The code of level k' in binade Eq is ((Eq + bias - 1) << M) + k' for normal and subnormal levels
// alike, and a carry to k' = 2^(M+1) lands on the first level of the next binade.
uint8_t sr_fp8_bits(uint32_t fbits, uint32_t r32, int e5m2) {
    const int M = e5m2 ? 2 : 3, bias = e5m2 ? 15 : 7;
    const uint32_t max_code = e5m2 ? 0x7Bu : 0x7Eu;
    const float max_value = e5m2 ? 57344.0f : 448.0f;
    const uint8_t sign = static_cast<uint8_t>((fbits >> 24) & 0x80u);
    if (is_nan_bits(fbits)) return 0x7F;
    const float a = float_of(fbits & 0x7FFFFFFFu);
    if (std::isinf(a)) return static_cast<uint8_t>(sign | (e5m2 ? 0x7Cu : max_code));
    if (a >= max_value) return static_cast<uint8_t>(sign | max_code);
    if (a == 0.0f) return sign;
    int E;
    std::frexp(a, &E);      // a = mant * 2^E with mant in [0.5, 1): binary exponent is E - 1
    E -= 1;
    const int Eq = E > 1 - bias ? E : 1 - bias;
    const double y = std::ldexp(static_cast<double>(a), M - Eq);      // exact: power-of-two scaling
    const double k = std::floor(y);
    const double f = y - k;
    const double threshold = std::floor(std::ldexp(f, 32));
    const uint32_t up = static_cast<double>(r32) < threshold ? 1u : 0u;
    uint32_t code = static_cast<uint32_t>((Eq + bias - 1) << M) + static_cast<uint32_t>(k) + up;
    if (code > max_code) code = max_code;
    return static_cast<uint8_t>(sign | code);
}

// 32 noise bits per element: one Philox call per four consecutive elements, counter number =
// index >> 2, element index & 3 takes output word index & 3 (key and the other counter words as above).
uint32_t noise32_for(uint64_t seed, uint32_t step, uint32_t tensor_id, uint64_t index) {
    const uint64_t number = index >> 2;
    const uint32_t ctr[4] = {static_cast<uint32_t>(number), static_cast<uint32_t>(number >> 32),
                             tensor_id, static_cast<uint32_t>(seed >> 32)};
    const uint32_t key[2] = {static_cast<uint32_t>(seed), step};
    uint32_t w[4];
    philox4x32_10(ctr, key, w);
    return w[index & 3u];
}

void oracle_sr_downcast_fp8(const float* src, uint8_t* dst, uint64_t n, int e5m2, uint64_t seed, uint32_t step,
                            uint32_t tensor_id, uint64_t elem_offset) {
#pragma omp parallel for schedule(static)
    for (int64_t i = 0; i < static_cast<int64_t>(n); ++i)
        dst[i] = sr_fp8_bits(bits_of(src[i]), noise32_for(seed, step, tensor_id, elem_offset + static_cast<uint64_t>(i)), e5m2);
}

uint8_t oracle_sr_fp8_bits(uint32_t fbits, uint32_t r32, int e5m2) { return sr_fp8_bits(fbits, r32, e5m2); }

uint32_t oracle_noise32(uint64_t seed, uint32_t step, uint32_t tensor_id, uint64_t index) {
    return noise32_for(seed, step, tensor_id, index);
}

// ---- Eq. 2 onto the 4-bit grid E2M1 ----------------------------------------------------------
// The same closing remark names 4-bit formats.  E2M1: one sign bit, 2 exponent bits (bias 1), one
// mantissa bit; the eight magnitudes are 0, 0.5, 1, 1.5, 2, 3, 4, 6 (codes 0..7); there is neither
// an infinity nor a NaN.  The rule is the one above with M = 1, bias = 1.  Every magnitude at or
// beyond 6 saturates to 6, infinity included; a NaN has no image in the format and is written as the
// largest magnitude with its sign bit (a choice of this restatement, not of the paper).
uint8_t sr_fp4_bits(uint32_t fbits, uint32_t r32) {
    const int M = 1, bias = 1;
    const uint32_t max_code = 7u;
    const uint8_t sign = static_cast<uint8_t>((fbits >> 28) & 0x8u);
    if (is_nan_bits(fbits)) return static_cast<uint8_t>(sign | max_code);
    const float a = float_of(fbits & 0x7FFFFFFFu);
    if (a >= 6.0f) return static_cast<uint8_t>(sign | max_code);
    if (a == 0.0f) return sign;
    int E;
    std::frexp(a, &E);
    E -= 1;
    const int Eq = E > 1 - bias ? E : 1 - bias;
    const double y = std::ldexp(static_cast<double>(a), M - Eq);
    const double k = std::floor(y);
    const double f = y - k;
    const double threshold = std::floor(std::ldexp(f, 32));
    const uint32_t up = static_cast<double>(r32) < threshold ? 1u : 0u;
    uint32_t code = static_cast<uint32_t>((Eq + bias - 1) << M) + static_cast<uint32_t>(k) + up;
    if (code > max_code) code = max_code;
    return static_cast<uint8_t>(sign | code);
}

uint8_t oracle_sr_fp4_bits(uint32_t fbits, uint32_t r32) { return sr_fp4_bits(fbits, r32); }

// Array form: two codes per byte, element 2j in bits 0..3 and element 2j+1 in bits 4..7 of byte j
// (the upper half of the last byte is 0 when n is odd).  Noise: the 32-bit word per element above.
void oracle_sr_downcast_fp4(const float* src, uint8_t* dst, uint64_t n, uint64_t seed, uint32_t step,
                            uint32_t tensor_id, uint64_t elem_offset) {
    const int64_t nbytes = static_cast<int64_t>((n + 1) / 2);
#pragma omp parallel for schedule(static)
    for (int64_t j = 0; j < nbytes; ++j) {
        const uint64_t i0 = 2u * static_cast<uint64_t>(j), i1 = i0 + 1;
        uint8_t b = sr_fp4_bits(bits_of(src[i0]), noise32_for(seed, step, tensor_id, elem_offset + i0));
        if (i1 < n)
            b = static_cast<uint8_t>(b | (sr_fp4_bits(bits_of(src[i1]), noise32_for(seed, step, tensor_id, elem_offset + i1)) << 4));
        dst[j] = b;
    }
}

// ---- Eq. 2 in a BF16 accumulation -------------------------------------------------------------
// Section 3 keeps every tensor in BF16, the accumulated gradient included.  Adding a small term to
// a BF16 accumulator with nearest rounding loses it whenever it is below half a spacing (the
// stagnation of Section 2.1); with Q_SR the expected sum is exact.  One accumulation:
//   t = scale * g          (FP32, one rounding; exact for scale = 1)
//   s = acc + t            (FP32, one rounding)
//   acc <- Q_SR(s)  or  Q(s)
// The noise is rounding slot 3 of the element's group (the counter number 4 * group + 3, which the
// optimizer step leaves unused), so that accumulation and update draw from disjoint streams even
// under the same (seed, step, tensor_id).
uint16_t accumulate_element(uint16_t acc, float g, float scale, uint32_t r16, int stochastic) {
    const float t = scale * g;
    const float s = bf16_to_float(acc) + t;
    return stochastic ? sr_bf16_bits(bits_of(s), r16) : rne_bf16_bits(bits_of(s));
}

uint16_t oracle_accumulate_element(uint16_t acc, float g, float scale, uint32_t r16, int stochastic) {
    return accumulate_element(acc, g, scale, r16, stochastic);
}

void oracle_sr_accumulate(uint16_t* acc, const void* g, int g_is_f32, uint64_t n, float scale, int stochastic,
                          uint64_t seed, uint32_t step, uint32_t tensor_id, uint64_t elem_offset) {
    const float* g32 = static_cast<const float*>(g);
    const uint16_t* g16 = static_cast<const uint16_t*>(g);
#pragma omp parallel for schedule(static)
    for (int64_t i = 0; i < static_cast<int64_t>(n); ++i) {
        const float gi = g_is_f32 ? g32[i] : bf16_to_float(g16[i]);
        const uint32_t r = noise_for_slot(seed, step, tensor_id, elem_offset + static_cast<uint64_t>(i), 3);
        acc[i] = accumulate_element(acc[i], gi, scale, r, stochastic);
    }
}

// Q_SR on an FP32 array; uses rounding slot 0 (the x slot) of the noise.
void oracle_sr_downcast(const float* src, uint16_t* dst, uint64_t n, uint64_t seed, uint32_t step,
                        uint32_t tensor_id, uint64_t elem_offset) {
#pragma omp parallel for schedule(static)
    for (int64_t i = 0; i < static_cast<int64_t>(n); ++i) {
        const uint32_t r = noise_for_slot(seed, step, tensor_id, elem_offset + static_cast<uint64_t>(i), 0);
        dst[i] = sr_bf16_bits(bits_of(src[i]), r);
    }
}

// ---- sum of squares with a fixed tree ------------------------------------------------------
// One reduction pass turns an array of L doubles into ceil(L/8192) doubles.  Inside a block of
// 8192 consecutive entries there are 256 accumulators; accumulator j adds, in this order, the
// entries  r*1024 + 4*j + k  for r = 0..7, k = 0..3  (entries past the end are skipped).  The 256
// accumulators form 8 groups of 32; each group is folded by a butterfly (partner = lane XOR 16,
// 8, 4, 2, 1; after it every lane of the group holds the same value) and the 8 group values are
// added in order 0..7.  Passes repeat until one value is left.  The first pass works on the
// squares g_i*g_i, which are exact in double for FP32 or BF16 g_i.
static double fold_block(const double* terms, uint64_t count) {
    double acc[256];
    for (int j = 0; j < 256; ++j) {
        double a = 0.0;
        for (int r = 0; r < 8; ++r)
            for (int k = 0; k < 4; ++k) {
                const uint64_t e = static_cast<uint64_t>(r) * 1024u + 4u * static_cast<uint64_t>(j) + static_cast<uint64_t>(k);
                if (e < count) a += terms[e];
            }
        acc[j] = a;
    }
    double group[8];
    for (int w = 0; w < 8; ++w) {
        double lane[32];
        for (int l = 0; l < 32; ++l) lane[l] = acc[32 * w + l];
        for (int s = 16; s >= 1; s >>= 1) {
            double next[32];
            for (int l = 0; l < 32; ++l) next[l] = lane[l] + lane[l ^ s];
            for (int l = 0; l < 32; ++l) lane[l] = next[l];
        }
        group[w] = lane[0];
    }
    double total = group[0];
    for (int w = 1; w < 8; ++w) total += group[w];
    return total;
}

double oracle_sqnorm(const void* g, int g_is_f32, uint64_t n) {
    if (n == 0) return 0.0;
    const uint16_t* g16 = static_cast<const uint16_t*>(g);
    const float* g32 = static_cast<const float*>(g);
    uint64_t count = (n + 8191u) / 8192u;
    double* level = new double[count];
#pragma omp parallel for schedule(static)
    for (int64_t c = 0; c < static_cast<int64_t>(count); ++c) {
        const uint64_t base = static_cast<uint64_t>(c) * 8192u;
        const uint64_t len = (n - base < 8192u) ? (n - base) : 8192u;
        double sq[8192];
        for (uint64_t e = 0; e < len; ++e) {
            const double gi = g_is_f32 ? static_cast<double>(g32[base + e])
                                       : static_cast<double>(bf16_to_float(g16[base + e]));
            sq[e] = gi * gi;
        }
        level[c] = fold_block(sq, len);
    }
    while (count > 1) {
        const uint64_t next_count = (count + 8191u) / 8192u;
        double* next = new double[next_count];
        for (uint64_t c = 0; c < next_count; ++c) {
            const uint64_t base = c * 8192u;
            const uint64_t len = (count - base < 8192u) ? (count - base) : 8192u;
            next[c] = fold_block(level + base, len);
        }
        delete[] level;
        level = next;
        count = next_count;
    }
    const double result = level[0];
    delete[] level;
    return result;
}

// Same tree applied to an array of doubles (used to check the later passes on their own).
double oracle_tree_sum(const double* terms, uint64_t n) {
    if (n == 0) return 0.0;
    uint64_t count = n;
    double* level = new double[count];
    std::memcpy(level, terms, count * sizeof(double));
    while (count > 1) {
        const uint64_t next_count = (count + 8191u) / 8192u;
        double* next = new double[next_count];
        for (uint64_t c = 0; c < next_count; ++c) {
            const uint64_t base = c * 8192u;
            const uint64_t len = (count - base < 8192u) ? (count - base) : 8192u;
            next[c] = fold_block(level + base, len);
        }
        delete[] level;
        level = next;
        count = next_count;
    }
    const double result = level[0];
    delete[] level;
    return result;
}

// Global-norm clipping with a gradient-accumulation factor: the true gradient is accum_scale * g,
// its norm is accum_scale * sqrt(S); the factor applied to g is accum_scale * min(1, max_norm /
// (norm + 1e-6)).  Evaluated in double, returned as FP32.
float oracle_clip_scale(double sqnorm, float accum_scale, float max_norm) {
    const double norm = static_cast<double>(accum_scale) * std::sqrt(sqnorm);
    double coef = static_cast<double>(max_norm) / (norm + 1e-6);
    if (coef > 1.0) coef = 1.0;
    return static_cast<float>(static_cast<double>(accum_scale) * coef);
}

}  // extern "C"
