// ECO oracle -- TEST INFRASTRUCTURE, NOT THE PRODUCT.
//
// A plain, slow, single-threaded CPU statement of the ECO quantized training
// step (Algorithm 1) with its two ECO_QUANTIZE forms (Algorithm 2 for momentum
// SGD, Algorithm 3 for Adam), the symmetric quantizer of Sec. 3.1
// ("Quantization") and the two rounding rules of the same section.  It exists
// only so that tests, the smoke check and the benchmark's CPU-baseline leg
// have something independent to compare the CUDA library with.  It shares no
// code, header, table or constant generator with the CUDA library and neither
// side includes the other.
//
// Every routine is templated on the real type R:
//   R = float   the arithmetic the CUDA kernels are compared with bit for bit
//               (one correctly rounded IEEE-754 binary32 operation per line;
//               std::fma is the only fused operation; compiled with
//               -ffp-contract=off so nothing else is contracted),
//   R = double  the same lines in binary64, used by the pins that check the
//               algebra of the paper (Lemma 3.5, Appendix A, Appendix C).
//
// Pins (tests/test_oracle_*.py): number-format tables against their closed
// form and a library cast; stochastic rounding probability by enumeration and
// by Monte Carlo; Philox against a library generator; identity quantizer ->
// plain SGDM / Adam; Lemma 3.5 telescoping; the Adam one-step identity;
// Appendix A exact equivalence with master weights; Appendix C stationary
// second moments of all three regimes (ECO, naive, master weights); the scale
// s = max|x| / rho by its consequences (the largest element of every block
// lands on +-rho, s * rho gives the maximum back) with block extents and code
// layout written out independently; power-of-two block scales against exact
// rational search, a library decode of the exponent byte and power-of-two
// invariance; the position of a row slice in the random stream against the
// whole tensor.  tests/test_oracle_mutations.py plants mistakes in a scratch
// copy of this file and checks that those pins fail.  The order of the
// binary32 operations is this build's choice (the paper fixes none): parity
// unpinned for that order alone.

#include <cmath>
#include <cstdint>
#include <cstring>
#include <limits>
#include <vector>

namespace {

// ---------------------------------------------------------------------------
// Enumerations of the boundary (values shared with the C-ABI by number only).
// ---------------------------------------------------------------------------
enum Format { FMT_FP8_E4M3 = 0, FMT_INT4 = 1, FMT_IDENTITY = 2, FMT_ADDITIVE_NOISE = 3, FMT_FP8_E5M2 = 4 };

bool is_fp8(int format) { return format == FMT_FP8_E4M3 || format == FMT_FP8_E5M2; }
enum Granularity { GRAN_TENSOR = 0, GRAN_ROW = 1, GRAN_BLOCK = 2 };
enum ScaleDtype { SCALE_NATIVE = 0, SCALE_BF16 = 1, SCALE_E8M0 = 2 };  // native = R; E8M0 = one byte, s = 2^(byte - 127)
enum Optimizer { OPT_SGDM = 0, OPT_ADAM = 1 };
enum Rounding { ROUND_RTN = 0, ROUND_SR = 1 };
enum Injection { INJECT_NONE = 0, INJECT_ECO = 1, INJECT_IDEAL = 2 };
enum GradDtype { GRAD_BF16 = 0, GRAD_NATIVE = 1 };

struct OracleConfig {
    int32_t format;
    int32_t granularity;
    int32_t block;        // B for GRAN_BLOCK
    int32_t scale_dtype;
    int32_t optimizer;
    int32_t rounding;
    int32_t injection;    // INJECT_ECO is the paper's method
    int32_t grad_dtype;
};

// ---------------------------------------------------------------------------
// Philox4x32-10 (Salmon, Moraes, Dror, Shaw, SC'11): counter-based generator.
// ---------------------------------------------------------------------------
void philox4x32_10(const uint32_t ctr[4], const uint32_t key[2], uint32_t out[4]) {
    const uint64_t M0 = 0xD2511F53u, M1 = 0xCD9E8D57u;  // round multipliers
    const uint32_t W0 = 0x9E3779B9u, W1 = 0xBB67AE85u;  // Weyl key increments
    uint32_t c0 = ctr[0], c1 = ctr[1], c2 = ctr[2], c3 = ctr[3];
    uint32_t k0 = key[0], k1 = key[1];
    for (int round = 0; round < 10; ++round) {
        const uint64_t p0 = M0 * c0;
        const uint64_t p1 = M1 * c2;
        const uint32_t n0 = static_cast<uint32_t>(p1 >> 32) ^ c1 ^ k0;
        const uint32_t n1 = static_cast<uint32_t>(p1);
        const uint32_t n2 = static_cast<uint32_t>(p0 >> 32) ^ c3 ^ k1;
        const uint32_t n3 = static_cast<uint32_t>(p0);
        c0 = n0; c1 = n1; c2 = n2; c3 = n3;
        k0 += W0; k1 += W1;
    }
    out[0] = c0; out[1] = c1; out[2] = c2; out[3] = c3;
}

// The random word of element i of tensor `tensor_id` at optimizer step `step`:
// key = seed, counter = (i / 4, tensor_id, step), word i mod 4.
uint32_t element_random_word(uint64_t seed, uint64_t step, uint32_t tensor_id, uint64_t i) {
    const uint32_t key[2] = {static_cast<uint32_t>(seed), static_cast<uint32_t>(seed >> 32)};
    const uint32_t ctr[4] = {static_cast<uint32_t>(i >> 2), tensor_id,
                             static_cast<uint32_t>(step), static_cast<uint32_t>(step >> 32)};
    uint32_t out[4];
    philox4x32_10(ctr, key, out);
    return out[i & 3];
}

// ---------------------------------------------------------------------------
// bfloat16 <-> binary32 (bf16 = the upper 16 bits of a binary32).
// ---------------------------------------------------------------------------
float bf16_to_f32(uint16_t h) {
    const uint32_t bits = static_cast<uint32_t>(h) << 16;
    float f;
    std::memcpy(&f, &bits, 4);
    return f;
}

uint16_t f32_to_bf16_rne(float f) {
    uint32_t bits;
    std::memcpy(&bits, &f, 4);
    if ((bits & 0x7FFFFFFFu) > 0x7F800000u) return static_cast<uint16_t>((bits >> 16) | 0x0040u);  // NaN
    const uint32_t lsb = (bits >> 16) & 1u;
    bits += 0x7FFFu + lsb;  // round to nearest, ties to even
    return static_cast<uint16_t>(bits >> 16);
}

// ---------------------------------------------------------------------------
// Number formats (Sec. 3.1: rho is the largest representable magnitude).
// FP8-E4M3 is the OCP "FN" flavour: 1 sign, 4 exponent (bias 7), 3 mantissa
// bits, no infinities, S.1111.111 is NaN, largest finite 448 = S.1111.110.
// INT4 is the symmetric integer grid -7..7 (two's complement nibble, -8 unused).
// FP8-E5M2 (the other OCP 8-bit float, offered as a further format on the same skeleton: Sec. 3.1 leaves the
// format open): 1 sign, 5 exponent (bias 15), 2 mantissa bits, IEEE-style infinities and NaNs (never written),
// largest finite 57344 = S.11110.11, subnormals M * 2^-16.
// ---------------------------------------------------------------------------
template <class R>
R format_rho(int format) {
    return format == FMT_FP8_E4M3 ? R(448) : (format == FMT_FP8_E5M2 ? R(57344) : R(7));
}

// Magnitude of a 7-bit E4M3 magnitude code (sign stripped).
template <class R>
R e4m3_magnitude(int mag_code) {
    const int E = (mag_code >> 3) & 15, M = mag_code & 7;
    if (E == 15 && M == 7) return std::numeric_limits<R>::quiet_NaN();
    if (E == 0) return std::ldexp(R(M), -9);                  // subnormal: M * 2^-9
    return std::ldexp(R(1) + R(M) / R(8), E - 7);             // 2^(E-7) * (1 + M/8)
}

// Magnitude of a 7-bit E5M2 magnitude code (sign stripped).
template <class R>
R e5m2_magnitude(int mag_code) {
    const int E = (mag_code >> 2) & 31, M = mag_code & 3;
    if (E == 31) return M == 0 ? std::numeric_limits<R>::infinity() : std::numeric_limits<R>::quiet_NaN();
    if (E == 0) return std::ldexp(R(M), -16);                 // subnormal: M * 2^-16
    return std::ldexp(R(1) + R(M) / R(4), E - 15);            // 2^(E-15) * (1 + M/4)
}

template <class R>
R code_value(int format, int code) {
    if (format == FMT_FP8_E5M2) {
        const R mag = e5m2_magnitude<R>(code & 0x7F);
        return (code & 0x80) ? -mag : mag;
    }
    if (format == FMT_FP8_E4M3) {
        const R mag = e4m3_magnitude<R>(code & 0x7F);
        return (code & 0x80) ? -mag : mag;
    }
    const int nib = code & 0xF;
    return R(nib >= 8 ? nib - 16 : nib);
}

// Lower grid neighbour (as a magnitude code) of a magnitude a in [0, rho] and
// the fraction of the gap above it.  All operations are exact in R.
template <class R>
void lower_neighbour(int format, R a, int* lo_code, R* frac) {
    if (format == FMT_INT4) {
        const R k = std::floor(a);
        *lo_code = static_cast<int>(k);
        *frac = a - k;
        return;
    }
    // binary floating-point grids: mb mantissa bits, smallest normal 2^emin, subnormal spacing 2^(emin - mb)
    const int mb = format == FMT_FP8_E5M2 ? 2 : 3;
    const int emin = format == FMT_FP8_E5M2 ? -14 : -6;
    if (a < std::ldexp(R(1), emin)) {
        const R q = std::ldexp(a, mb - emin);
        const R k = std::floor(q);
        *lo_code = static_cast<int>(k);
        *frac = q - k;
        return;
    }
    int ex;
    std::frexp(a, &ex);                       // a = f * 2^ex, f in [0.5, 1)
    const int e = ex - 1;                     // 2^e <= a < 2^(e+1)
    const R q = std::ldexp(a, mb - e);        // in [2^mb, 2^(mb+1)): spacing 2^(e-mb)
    const R k = std::floor(q);
    *lo_code = ((e - emin + 1) << mb) | (static_cast<int>(k) - (1 << mb));
    *frac = q - k;
}

// Round a scaled value y = x / s to a code of the format (Sec. 3.1, rounding
// paragraph).  Magnitudes beyond rho are clamped to rho first; a NaN takes +rho
// whatever its sign bit (IEEE 754 leaves the sign of a computed NaN open, and processors differ).
//   RTN: the closest grid point, ties to the even code.
//   SR : the upper neighbour with probability frac (the distance to the lower
//        one over the gap), decided by comparing the top 24 bits of the
//        element's random word with frac * 2^24.
template <class R>
int round_to_code(int format, int rounding, R y, uint32_t random_word) {
    const R rho = format_rho<R>(format);
    const bool negative = std::signbit(y) && !std::isnan(y);   // the sign bit of a NaN means nothing: it takes +rho
    const R ay = std::fabs(y);
    const R a = (ay < rho) ? ay : rho;
    int lo;
    R frac;
    lower_neighbour<R>(format, a, &lo, &frac);
    bool up;
    if (rounding == ROUND_SR) {
        const R u = R(random_word >> 8);
        up = u < frac * R(16777216);
    } else {
        up = (frac > R(0.5)) || (frac == R(0.5) && (lo & 1));
    }
    const int mag = lo + (up ? 1 : 0);
    if (is_fp8(format)) return (negative ? 0x80 : 0) | mag;
    return (negative ? -mag : mag) & 0xF;
}

// ---------------------------------------------------------------------------
// Storage helpers: codes (one byte per FP8 element; two INT4 elements per
// byte, element 2k in the low nibble) and scales (R, or bf16 when R = float).
// ---------------------------------------------------------------------------
int load_code(int format, const uint8_t* w, uint64_t i) {
    if (is_fp8(format)) return w[i];
    const uint8_t byte = w[i >> 1];
    return (i & 1) ? (byte >> 4) : (byte & 0xF);
}

void store_code(int format, uint8_t* w, uint64_t i, int code) {
    if (is_fp8(format)) { w[i] = static_cast<uint8_t>(code); return; }
    uint8_t& byte = w[i >> 1];
    if (i & 1) byte = static_cast<uint8_t>((byte & 0x0F) | ((code & 0xF) << 4));
    else       byte = static_cast<uint8_t>((byte & 0xF0) | (code & 0xF));
}

template <class R>
R load_scale(int scale_dtype, const void* scale, uint64_t k) {
    if (scale_dtype == SCALE_BF16) return R(bf16_to_f32(static_cast<const uint16_t*>(scale)[k]));
    if (scale_dtype == SCALE_E8M0) return std::ldexp(R(1), static_cast<int>(static_cast<const uint8_t*>(scale)[k]) - 127);
    return static_cast<const R*>(scale)[k];
}

// Power-of-two scale (the shared-exponent scales of microscaling formats, which Sec. 3.1 cites among the group-wise
// schemes): the smallest power of two s with s * rho >= amax, so that, like s = max|x| / rho, it prevents overflow;
// exponent kept within what one byte with bias 127 holds (-127 .. 127; 0xFF is never written).
template <class R>
int pow2_scale_exponent(R amax, R rho) {
    int e;
    std::frexp(static_cast<long double>(amax / rho), &e);      // a first guess; the loops below decide exactly
    if (e > 127) e = 127;
    if (e < -127) e = -127;
    const long double a = static_cast<long double>(amax), r = static_cast<long double>(rho);
    while (e < 127 && std::ldexp(r, e) < a) ++e;
    while (e > -127 && std::ldexp(r, e - 1) >= a) --e;
    return e;
}

// Scale of a block with maximum magnitude amax (Sec. 3.1: s = max|x| / rho).
// Returns the stored scale s and the factor `inv` that maps values onto the
// code grid (rho / max|x|, i.e. the paper's round(rho x / max|x|); with a
// bf16 scale the grid is the one the rounded scale defines, 1 / s).
// An all-zero block takes s = 1.
template <class R>
void make_scale(int format, int scale_dtype, R amax, void* scale, uint64_t k, R* s_out, R* inv_out) {
    const R rho = format_rho<R>(format);
    R s, inv;
    if (amax == R(0)) {
        s = R(1);
        inv = R(1);
        if (scale_dtype == SCALE_BF16) static_cast<uint16_t*>(scale)[k] = f32_to_bf16_rne(1.0f);
        else if (scale_dtype == SCALE_E8M0) static_cast<uint8_t*>(scale)[k] = 127;
        else static_cast<R*>(scale)[k] = s;
    } else if (scale_dtype == SCALE_E8M0) {
        const int e = pow2_scale_exponent<R>(amax, rho);
        static_cast<uint8_t*>(scale)[k] = static_cast<uint8_t>(e + 127);
        s = std::ldexp(R(1), e);
        inv = std::ldexp(R(1), -e);
    } else if (scale_dtype == SCALE_BF16) {
        const uint16_t h = f32_to_bf16_rne(static_cast<float>(amax / rho));
        static_cast<uint16_t*>(scale)[k] = h;
        s = R(bf16_to_f32(h));
        inv = R(1) / s;
    } else {
        s = amax / rho;
        inv = rho / amax;
        static_cast<R*>(scale)[k] = s;
    }
    *s_out = s;
    *inv_out = inv;
}

// Extent of the scale blocks of a [rows, cols] row-major tensor.
struct BlockGrid {
    uint64_t n_blocks;       // number of scale blocks
    uint64_t blocks_per_row; // GRAN_BLOCK only
};

BlockGrid block_grid(const OracleConfig& cfg, uint64_t rows, uint64_t cols) {
    BlockGrid g{1, 1};
    if (cfg.granularity == GRAN_ROW) g.n_blocks = rows;
    if (cfg.granularity == GRAN_BLOCK) {
        g.blocks_per_row = (cols + cfg.block - 1) / cfg.block;
        g.n_blocks = rows * g.blocks_per_row;
    }
    return g;
}

// First element (row-major index) and length of scale block k.
void block_extent(const OracleConfig& cfg, const BlockGrid& g, uint64_t rows, uint64_t cols,
                  uint64_t k, uint64_t* begin, uint64_t* len) {
    if (cfg.granularity == GRAN_TENSOR) { *begin = 0; *len = rows * cols; return; }
    if (cfg.granularity == GRAN_ROW) { *begin = k * cols; *len = cols; return; }
    const uint64_t row = k / g.blocks_per_row, j = k % g.blocks_per_row;
    const uint64_t c0 = j * cfg.block;
    *begin = row * cols + c0;
    *len = (cols - c0 < static_cast<uint64_t>(cfg.block)) ? cols - c0 : cfg.block;
}

// ---------------------------------------------------------------------------
// q(x): the symmetric quantizer of Sec. 3.1 applied block by block.  Used for
// the initial state theta_hat_0 = q(theta_0) (Appendix A, initialisation) and
// by the master-weight reference of the tests.
// index_base: position of x[0] inside the full tensor when x is a slice of whole rows of it (0 for a
// whole tensor); the random word of element i is the one of position index_base + i, so a slice
// rounds exactly like the same rows inside the whole tensor.
// ---------------------------------------------------------------------------
template <class R>
int quantize_tensor(const OracleConfig& cfg, const R* x, uint64_t rows, uint64_t cols,
                    uint8_t* w, void* scale, uint64_t seed, uint64_t step, uint32_t tensor_id,
                    uint64_t index_base) {
    const BlockGrid g = block_grid(cfg, rows, cols);
    for (uint64_t k = 0; k < g.n_blocks; ++k) {
        uint64_t begin, len;
        block_extent(cfg, g, rows, cols, k, &begin, &len);
        R amax = R(0);
        for (uint64_t i = begin; i < begin + len; ++i) {
            const R ax = std::fabs(x[i]);
            if (ax > amax) amax = ax;
        }
        R s, inv;
        make_scale<R>(cfg.format, cfg.scale_dtype, amax, scale, k, &s, &inv);
        for (uint64_t i = begin; i < begin + len; ++i) {
            const uint32_t r = cfg.rounding == ROUND_SR ? element_random_word(seed, step, tensor_id, index_base + i) : 0u;
            store_code(cfg.format, w, i, round_to_code<R>(cfg.format, cfg.rounding, x[i] * inv, r));
        }
    }
    return 0;
}

template <class R>
int dequantize_tensor(const OracleConfig& cfg, const uint8_t* w, const void* scale,
                      uint64_t rows, uint64_t cols, R* x) {
    const BlockGrid g = block_grid(cfg, rows, cols);
    for (uint64_t k = 0; k < g.n_blocks; ++k) {
        uint64_t begin, len;
        block_extent(cfg, g, rows, cols, k, &begin, &len);
        const R s = load_scale<R>(cfg.scale_dtype, scale, k);
        for (uint64_t i = begin; i < begin + len; ++i)
            x[i] = code_value<R>(cfg.format, load_code(cfg.format, w, i)) * s;
    }
    return 0;
}

// ---------------------------------------------------------------------------
// Hyper-parameters H and the scalars derived from them once per step, in
// binary64, each cast to R once.
// ---------------------------------------------------------------------------
struct Hyper {
    double lr, beta1, beta2, eps;
    uint64_t step;  // t, 1-based: the count of updates including this one
    uint64_t seed;
    // The two ingredients every experiment of Sec. 4 adds to OPTIM_STEP ("AdamW ... weight decay of
    // 0.1 and gradient clipping with a norm of 1.0") and that Algorithms 1-3 leave inside the optimizer's
    // step function: decoupled weight decay lambda, and one global factor on the gradient (the clipping
    // factor min(1, c / ||g||), computed by the caller).  0 and 1 switch them off.
    double weight_decay = 0.0;
    double grad_scale = 1.0;
    // Position of the buffers' first element inside the full tensor when they hold a slice of whole rows of it
    // (0 for a whole tensor): element i draws the random word of position index_base + i.
    uint64_t index_base = 0;
};

template <class R>
struct StepScalars {
    R beta1, beta2, eps;
    R one_minus_beta1, one_minus_beta2;
    R neg_lr;          // SGDM: theta~ = theta^ - eta m~            (Eq. theta_tilde)
    R neg_lr_wd;       // decoupled decay: theta^ <- theta^ - (eta lambda) theta^
    R grad_scale;      // g <- grad_scale * g
    bool decay;
    R alpha;           // SGDM: (1/eta)(1 - 1/beta)                 (Eq. alpha)
    R inv_lr;          // ideal injection (Appendix A): 1/eta
    R inv_lr_beta;     // ideal injection (Appendix A): 1/(eta beta)
    R inv_bc2;         // Adam: 1 / (1 - beta2^t)
    R lr_over_bc1;     // Adam: eta / (1 - beta1^t)
    R adam_coef;       // Adam: ((1 - beta1^t)/eta)(1 - 1/beta1)    (Algorithm 3, line 5)
};

template <class R>
StepScalars<R> derive_scalars(const Hyper& h) {
    StepScalars<R> s;
    const double t = static_cast<double>(h.step);
    const double bc1 = 1.0 - std::pow(h.beta1, t);
    const double bc2 = 1.0 - std::pow(h.beta2, t);
    s.beta1 = R(h.beta1);
    s.beta2 = R(h.beta2);
    s.eps = R(h.eps);
    s.one_minus_beta1 = R(1.0 - h.beta1);
    s.one_minus_beta2 = R(1.0 - h.beta2);
    s.neg_lr = R(-h.lr);
    s.neg_lr_wd = R(-(h.lr * h.weight_decay));
    s.grad_scale = R(h.grad_scale);
    s.decay = h.weight_decay != 0.0;
    s.alpha = R((1.0 / h.lr) * (1.0 - 1.0 / h.beta1));
    s.inv_lr = R(1.0 / h.lr);
    s.inv_lr_beta = R(1.0 / (h.lr * h.beta1));
    s.inv_bc2 = R(1.0 / bc2);
    s.lr_over_bc1 = R(h.lr / bc1);
    s.adam_coef = R((bc1 / h.lr) * (1.0 - 1.0 / h.beta1));
    return s;
}

// ---------------------------------------------------------------------------
// Algorithm 1 for one tensor: OPTIM_STEP on the dequantized weights, then
// ECO_QUANTIZE (Algorithm 2 or 3), scale block by scale block.
//
//   w, scale   in/out  quantized weights theta^ and their scales
//              (FMT_IDENTITY / FMT_ADDITIVE_NOISE: w is an R array, no scales)
//   grad       in      gradient, bf16 bit patterns or R
//   m, v       in/out  first / second moment (v unused by SGDM)
//   noise      in      FMT_ADDITIVE_NOISE only: xi, so that q(x) = x + xi
//   e_prev     in/out  INJECT_IDEAL only: the stored residual e_t (Appendix A)
//   dbg_theta_tilde, dbg_err   out, optional: theta~_{t+1} and e_{t+1}
// ---------------------------------------------------------------------------
template <class R>
int step_tensor(const OracleConfig& cfg, const Hyper& hyper,
                void* w, void* scale, const void* grad, R* m, R* v,
                uint64_t rows, uint64_t cols, uint32_t tensor_id,
                const R* noise, R* e_prev, R* dbg_theta_tilde, R* dbg_err) {
    const StepScalars<R> sc = derive_scalars<R>(hyper);
    const bool coded = is_fp8(cfg.format) || cfg.format == FMT_INT4;
    OracleConfig grid_cfg = cfg;
    if (!coded) grid_cfg.granularity = GRAN_TENSOR;
    const BlockGrid g = block_grid(grid_cfg, rows, cols);
    std::vector<R> theta_tilde, m_tilde, denom;

    for (uint64_t k = 0; k < g.n_blocks; ++k) {
        uint64_t begin, len;
        block_extent(grid_cfg, g, rows, cols, k, &begin, &len);
        theta_tilde.resize(len);
        m_tilde.resize(len);
        if (cfg.optimizer == OPT_ADAM) denom.resize(len);

        // ---- Algorithm 1, line 1: OPTIM_STEP on theta^_t ------------------
        const R s_old = coded ? load_scale<R>(cfg.scale_dtype, scale, k) : R(1);
        R amax = R(0);
        for (uint64_t j = 0; j < len; ++j) {
            const uint64_t i = begin + j;
            const R graw = cfg.grad_dtype == GRAD_BF16
                               ? R(bf16_to_f32(static_cast<const uint16_t*>(grad)[i]))
                               : static_cast<const R*>(grad)[i];
            const R gi = graw * sc.grad_scale;                                      // clipped / unscaled gradient
            R th = coded ? code_value<R>(cfg.format, load_code(cfg.format, static_cast<const uint8_t*>(w), i)) * s_old
                         : static_cast<const R*>(w)[i];
            if (sc.decay) th = std::fma(sc.neg_lr_wd, th, th);                      // AdamW: theta (1 - eta lambda)
            R tht;
            const R mt = std::fma(sc.beta1, m[i], sc.one_minus_beta1 * gi);          // Eq. m_tilde
            if (cfg.optimizer == OPT_SGDM) {
                tht = std::fma(sc.neg_lr, mt, th);                                  // Eq. theta_tilde
            } else {
                const R vt = std::fma(sc.beta2, v[i], sc.one_minus_beta2 * (gi * gi));
                const R den = std::sqrt(vt * sc.inv_bc2) + sc.eps;                  // sqrt(v/(1-b2^t)) + eps
                const R upd = (sc.lr_over_bc1 * mt) / den;                          // eta (m/(1-b1^t)) / den
                tht = th - upd;
                v[i] = vt;                                                          // Algorithm 3 returns v unchanged
                denom[j] = den;
            }
            theta_tilde[j] = tht;
            m_tilde[j] = mt;
            const R at = std::fabs(tht);
            if (at > amax) amax = at;
        }

        // ---- Algorithm 2 / 3 ----------------------------------------------
        R s = R(1), inv = R(1);
        if (coded) make_scale<R>(cfg.format, cfg.scale_dtype, amax, scale, k, &s, &inv);
        for (uint64_t j = 0; j < len; ++j) {
            const uint64_t i = begin + j;
            const R tht = theta_tilde[j];
            // line 1: theta^_{t+1} = q(theta~_{t+1})
            R thq;
            if (coded) {
                const uint32_t r = cfg.rounding == ROUND_SR
                                       ? element_random_word(hyper.seed, hyper.step, tensor_id, hyper.index_base + i) : 0u;
                const int code = round_to_code<R>(cfg.format, cfg.rounding, tht * inv, r);
                store_code(cfg.format, static_cast<uint8_t*>(w), i, code);
                thq = code_value<R>(cfg.format, code) * s;
            } else {
                thq = cfg.format == FMT_ADDITIVE_NOISE ? tht + noise[i] : tht;
                static_cast<R*>(w)[i] = thq;
            }
            // line 2: e_{t+1} = theta~_{t+1} - theta^_{t+1}
            const R e = tht - thq;
            // line 5: inject into the momentum
            const R mt = m_tilde[j];
            R mh = mt;
            if (cfg.injection == INJECT_ECO) {
                if (cfg.optimizer == OPT_SGDM) mh = std::fma(sc.alpha, e, mt);                 // Eq. m_hat
                else                           mh = std::fma(sc.adam_coef * denom[j], e, mt);  // Algorithm 3, line 5
            } else if (cfg.injection == INJECT_IDEAL) {
                // Appendix A: m <- m_bar + e_t / eta - e_{t+1} / (eta beta)
                mh = mt + sc.inv_lr * e_prev[i] - sc.inv_lr_beta * e;
                e_prev[i] = e;
            }
            m[i] = mh;
            if (dbg_theta_tilde) dbg_theta_tilde[i] = tht;
            if (dbg_err) dbg_err[i] = e;
        }
    }
    return 0;
}

}  // namespace

// ---------------------------------------------------------------------------
// C entry points for the ctypes binding in oracle/__init__.py.
// ---------------------------------------------------------------------------
extern "C" {

void eco_oracle_philox4x32_10(const uint32_t* ctr, const uint32_t* key, uint32_t* out) {
    philox4x32_10(ctr, key, out);
}

uint32_t eco_oracle_element_random_word(uint64_t seed, uint64_t step, uint32_t tensor_id, uint64_t i) {
    return element_random_word(seed, step, tensor_id, i);
}

double eco_oracle_code_value(int format, int code) { return code_value<double>(format, code); }

// Round n already-scaled values with explicit random words.
void eco_oracle_round_f32(int format, int rounding, const float* y, const uint32_t* r, uint64_t n, uint8_t* codes) {
    for (uint64_t i = 0; i < n; ++i) codes[i] = static_cast<uint8_t>(round_to_code<float>(format, rounding, y[i], r ? r[i] : 0u));
}
void eco_oracle_round_f64(int format, int rounding, const double* y, const uint32_t* r, uint64_t n, uint8_t* codes) {
    for (uint64_t i = 0; i < n; ++i) codes[i] = static_cast<uint8_t>(round_to_code<double>(format, rounding, y[i], r ? r[i] : 0u));
}

uint16_t eco_oracle_f32_to_bf16(float f) { return f32_to_bf16_rne(f); }

int eco_oracle_quantize_f32(const OracleConfig* cfg, const float* x, uint64_t rows, uint64_t cols,
                            uint8_t* w, void* scale, uint64_t seed, uint64_t step, uint32_t tensor_id,
                            uint64_t index_base) {
    return quantize_tensor<float>(*cfg, x, rows, cols, w, scale, seed, step, tensor_id, index_base);
}
int eco_oracle_quantize_f64(const OracleConfig* cfg, const double* x, uint64_t rows, uint64_t cols,
                            uint8_t* w, void* scale, uint64_t seed, uint64_t step, uint32_t tensor_id,
                            uint64_t index_base) {
    return quantize_tensor<double>(*cfg, x, rows, cols, w, scale, seed, step, tensor_id, index_base);
}
int eco_oracle_dequantize_f32(const OracleConfig* cfg, const uint8_t* w, const void* scale,
                              uint64_t rows, uint64_t cols, float* x) {
    return dequantize_tensor<float>(*cfg, w, scale, rows, cols, x);
}
int eco_oracle_dequantize_f64(const OracleConfig* cfg, const uint8_t* w, const void* scale,
                              uint64_t rows, uint64_t cols, double* x) {
    return dequantize_tensor<double>(*cfg, w, scale, rows, cols, x);
}

int eco_oracle_step_f32(const OracleConfig* cfg, double lr, double beta1, double beta2, double eps,
                        uint64_t step, uint64_t seed,
                        void* w, void* scale, const void* grad, float* m, float* v,
                        uint64_t rows, uint64_t cols, uint32_t tensor_id,
                        const float* noise, float* e_prev, float* dbg_theta_tilde, float* dbg_err, uint64_t index_base) {
    Hyper h{lr, beta1, beta2, eps, step, seed};
    h.index_base = index_base;
    return step_tensor<float>(*cfg, h, w, scale, grad, m, v, rows, cols, tensor_id,
                              noise, e_prev, dbg_theta_tilde, dbg_err);
}
int eco_oracle_step_ex_f32(const OracleConfig* cfg, double lr, double beta1, double beta2, double eps,
                           double weight_decay, double grad_scale, uint64_t step, uint64_t seed,
                           void* w, void* scale, const void* grad, float* m, float* v,
                           uint64_t rows, uint64_t cols, uint32_t tensor_id, uint64_t index_base) {
    Hyper h{lr, beta1, beta2, eps, step, seed};
    h.index_base = index_base;
    h.weight_decay = weight_decay;
    h.grad_scale = grad_scale;
    return step_tensor<float>(*cfg, h, w, scale, grad, m, v, rows, cols, tensor_id, nullptr, nullptr, nullptr, nullptr);
}
int eco_oracle_step_ex_f64(const OracleConfig* cfg, double lr, double beta1, double beta2, double eps,
                           double weight_decay, double grad_scale, uint64_t step, uint64_t seed,
                           void* w, void* scale, const void* grad, double* m, double* v,
                           uint64_t rows, uint64_t cols, uint32_t tensor_id, uint64_t index_base) {
    Hyper h{lr, beta1, beta2, eps, step, seed};
    h.index_base = index_base;
    h.weight_decay = weight_decay;
    h.grad_scale = grad_scale;
    return step_tensor<double>(*cfg, h, w, scale, grad, m, v, rows, cols, tensor_id, nullptr, nullptr, nullptr, nullptr);
}
int eco_oracle_step_f64(const OracleConfig* cfg, double lr, double beta1, double beta2, double eps,
                        uint64_t step, uint64_t seed,
                        void* w, void* scale, const void* grad, double* m, double* v,
                        uint64_t rows, uint64_t cols, uint32_t tensor_id,
                        const double* noise, double* e_prev, double* dbg_theta_tilde, double* dbg_err, uint64_t index_base) {
    Hyper h{lr, beta1, beta2, eps, step, seed};
    h.index_base = index_base;
    return step_tensor<double>(*cfg, h, w, scale, grad, m, v, rows, cols, tensor_id,
                               noise, e_prev, dbg_theta_tilde, dbg_err);
}

}  // extern "C"
