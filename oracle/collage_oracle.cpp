// CPU oracle for the Collage bf16 multi-component-float (MCF) AdamW step.
//
// TEST INFRASTRUCTURE ONLY.  This file is the slow, plain, obviously-correct
// restatement of what the optimizer step computes.  It shares no code, header,
// table or helper with the CUDA library and must never be reachable from the
// product path; only the tests, the smoke check and the benchmark's CPU
// baseline leg may load it.
//
// Arithmetic model (Section 3.1, "F^BF16(a op b)"; footnote of Section 4.1 on
// round-to-nearest): every written operator takes bfloat16 operands, forms
// the real result, and rounds ONCE to the nearest bfloat16, ties to even.
// Realisation here: operands are widened to double (exact), the operation is
// done in double, and the double is rounded to bfloat16 by the software
// rounder below.  A product of two bfloat16 values has at most 16 significant
// bits and is exact in double; for + - / sqrt the intermediate 53-bit rounding
// is innocuous because 53 >= 2*8+2.
//
// bfloat16 = 1 sign, 8 exponent, 7 stored mantissa bits, ulp(1) = 2^-7
// (Appendix A, table of formats); gradual underflow, overflow to infinity.
//
// Parity pins for every function are in tests/test_oracle_*.py.  Functions
// whose reading the paper does not fix (epsilon placement, the operand of the
// weight-decay product, the order of rounded operations inside one printed
// expression, the Kahan and float comparators) are marked "reading" below:
// parity unpinned by the paper for those choices -- they are pinned only through
// closed forms, exact rationals and the fp64 AdamW bound, not by a value the
// paper prints.  The lost count (Def. 3.2, Figure 3 left) follows the value
// of the parameter and is pinned against exact rationals on cases where the
// other candidate reading (stored components) gives a different count.

#include <cmath>
#include <cstdint>
#include <cstring>
#include <vector>
#include <algorithm>
#ifdef _OPENMP
#include <omp.h>
#endif

namespace {

typedef uint16_t bf16;

// ---------------------------------------------------------------- format ---

inline double widen(bf16 h) {
    uint32_t u = static_cast<uint32_t>(h) << 16;
    float f;
    std::memcpy(&f, &u, sizeof f);
    return static_cast<double>(f);
}

// Round a double to the nearest bfloat16, ties to even (Section 3.1; Def. 3.1
// for the spacing).  Works on the value, not on the bit pattern of a float:
// |x| = n * q with q = 2^(max(E,-126) - 7) the spacing at x's binade, n is
// rounded to an integer, and the integer is re-encoded.
bf16 round_to_bf16(double x) {
    const bf16 sign = std::signbit(x) ? 0x8000u : 0u;
    if (std::isnan(x)) return 0x7FC0u;
    if (std::isinf(x)) return sign | 0x7F80u;
    const double ax = std::fabs(x);
    if (ax == 0.0) return sign;
    int e2;
    std::frexp(ax, &e2);            // ax = f * 2^e2, f in [0.5, 1)
    int E = e2 - 1;                 // 2^E <= ax < 2^(E+1)
    if (E < -126) E = -126;         // subnormal binade shares the spacing of 2^-126
    const double n = std::ldexp(ax, -(E - 7));   // exact scaling
    double fl = std::floor(n);
    const double frac = n - fl;                  // exact, in [0,1)
    if (frac > 0.5 || (frac == 0.5 && std::fmod(fl, 2.0) == 1.0)) fl += 1.0;
    long r = static_cast<long>(fl);              // 0 .. 256
    if (r == 256) { r = 128; E += 1; }           // carry into the next binade
    if (r < 128) return sign | static_cast<bf16>(r);          // subnormal (E == -126) or zero
    const int field = E + 127;
    if (field >= 255) return sign | 0x7F80u;                  // overflow
    return sign | static_cast<bf16>((field << 7) | (r - 128));
}

// One rounded bfloat16 operation each (Section 3.1 notation).
inline bf16 op_add(bf16 a, bf16 b) { return round_to_bf16(widen(a) + widen(b)); }
inline bf16 op_sub(bf16 a, bf16 b) { return round_to_bf16(widen(a) - widen(b)); }
inline bf16 op_mul(bf16 a, bf16 b) { return round_to_bf16(widen(a) * widen(b)); }
inline bf16 op_div(bf16 a, bf16 b) { return round_to_bf16(widen(a) / widen(b)); }
inline bf16 op_sqrt(bf16 a)        { return round_to_bf16(std::sqrt(widen(a))); }
// a*b + c with a single rounding ("in FMA", Algorithm TwoProdFMA).  The product is exact in
// double; the sum p + c may need far more than 53 bits (a huge product and a tiny addend that only
// breaks a tie), so it is rounded to odd first: the double keeps a sticky last bit, which makes
// the final rounding to 8 bits the single rounding of the exact value.
inline bf16 op_fma(bf16 a, bf16 b, bf16 c) {
    const double p = widen(a) * widen(b);
    const double q = widen(c);
    double s = p + q;
    if (std::isfinite(s) && std::isfinite(p) && std::isfinite(q)) {
        const double qv = s - p;
        const double err = (p - (s - qv)) + (q - qv);      // TwoSum: p + q = s + err exactly
        if (err != 0.0) {
            uint64_t bits;
            std::memcpy(&bits, &s, sizeof bits);
            if ((bits & 1u) == 0)                           // even: step to the odd neighbour on err's side
                s = std::nextafter(s, err > 0.0 ? INFINITY : -INFINITY);
        }
    }
    return round_to_bf16(s);
}
inline bf16 op_neg(bf16 a) { return a ^ 0x8000u; }

struct pair16 { bf16 hi, lo; };

// ------------------------------------------------- basic MCF algorithms ---

// Theorem 4.1 (Fast2Sum): x = F(a+b); y = F(b - F(x-a)).  No sorting is done;
// exactness holds when |a| >= |b|.
inline pair16 fast_two_sum(bf16 a, bf16 b) {
    const bf16 x = op_add(a, b);
    const bf16 y = op_sub(b, op_sub(x, a));
    return {x, y};
}

// Algorithm TwoSum (Appendix C): six operations, no ordering requirement.
inline pair16 two_sum(bf16 a, bf16 b) {
    const bf16 x = op_add(a, b);
    const bf16 b_virtual = op_sub(x, a);
    const bf16 a_virtual = op_sub(x, b_virtual);
    const bf16 b_roundoff = op_sub(b, b_virtual);
    const bf16 a_roundoff = op_sub(a, a_virtual);
    return {x, op_add(a_roundoff, b_roundoff)};
}

// Algorithm TwoProdFMA: x = F(a*b); e = F(a*b - x) fused.
inline pair16 two_prod_fma(bf16 a, bf16 b) {
    const bf16 x = op_mul(a, b);
    return {x, op_fma(a, b, op_neg(x))};
}

// Algorithm Split (Veltkamp).  The constant is 2^c + 1 with c = 4 for the
// 8-bit significand (7 stored + hidden bit); with c = 3 the Dekker product
// below no longer reproduces TwoProdFMA.
inline pair16 split(bf16 a) {
    const bf16 factor = round_to_bf16(17.0);
    const bf16 t = op_mul(factor, a);
    const bf16 hi = op_sub(t, op_sub(t, a));
    return {hi, op_sub(a, hi)};
}

// Algorithm TwoProd (Dekker, no FMA).  The printed line subtracts from an
// undefined "p"; it is the product x.
inline pair16 two_prod_dekker(bf16 a, bf16 b) {
    const bf16 x = op_mul(a, b);
    const pair16 sa = split(a), sb = split(b);
    const bf16 err1 = op_sub(x, op_mul(sa.hi, sb.hi));
    const bf16 err2 = op_sub(err1, op_mul(sa.lo, sb.hi));
    const bf16 err3 = op_sub(err2, op_mul(sa.hi, sb.lo));
    return {x, op_sub(op_mul(sa.lo, sb.lo), err3)};
}

// Algorithm 1 (Grow): add a float a to the expansion (x, y).
inline pair16 grow(pair16 xy, bf16 a) {
    pair16 uv = fast_two_sum(xy.hi, a);
    return fast_two_sum(uv.hi, op_add(xy.lo, uv.lo));
}

// Algorithm Scaling: float v times expansion (a1, a2).  Every circled
// operator of the printed line rounds (reading).
inline pair16 scaling(bf16 v, pair16 a) {
    pair16 xe = two_prod_fma(a.hi, v);
    const bf16 e = op_add(op_mul(a.lo, v), xe.lo);
    return fast_two_sum(xe.hi, e);
}

// Algorithm Mul: expansion (a1, a2) times expansion (b1, b2).  Every circled
// operator of the printed line rounds (reading).
inline pair16 mul(pair16 a, pair16 b) {
    pair16 xe = two_prod_fma(a.hi, b.hi);
    const bf16 cross = op_add(op_mul(a.hi, b.lo), op_mul(a.lo, b.hi));
    const bf16 e = op_add(xe.lo, cross);
    return fast_two_sum(xe.hi, e);
}

// Renormalize is named by the paper's listing keywords but never defined; for
// a length-2 expansion it is Fast2Sum(hi, lo) (reading).
inline pair16 renormalize(pair16 a) { return fast_two_sum(a.hi, a.lo); }

// ------------------------------------------------------------- scalars ---

struct scalars {
    bf16 b1, c1, b2, c2, b2h, b2l, bc1, bc2, a, lam, eps;
};

// Algorithm 2 line 1, Table 1 (beta2 expansions) and Appendix D "Scalar and
// Bias Correction": every scalar expression is evaluated in double and only
// then cast to bfloat16.
scalars derive_scalars(double lr, double beta1, double beta2, double eps, double wd, uint64_t t) {
    scalars s;
    s.b1 = round_to_bf16(beta1);
    s.c1 = round_to_bf16(1.0 - beta1);
    s.b2 = round_to_bf16(beta2);
    s.c2 = round_to_bf16(1.0 - beta2);
    s.b2h = s.b2;
    s.b2l = round_to_bf16(beta2 - widen(s.b2h));
    s.bc1 = round_to_bf16(1.0 - std::pow(beta1, static_cast<double>(t)));
    s.bc2 = round_to_bf16(1.0 - std::pow(beta2, static_cast<double>(t)));
    s.a = round_to_bf16(lr);
    s.lam = round_to_bf16(wd);
    s.eps = round_to_bf16(eps);
    return s;
}

enum { STRAT_BF16 = 0, STRAT_LIGHT = 1, STRAT_PLUS = 2, STRAT_KAHAN = 3 };
enum { FLAG_EPS_INSIDE_SQRT = 1, FLAG_TWOSUM_GROW = 2, FLAG_DECAY_BY_GROW = 4 };

// Grow with TwoSum in place of Fast2Sum (Appendix C: TwoSum yields the same expansion for any
// a, b without sorting): exact also where |x| < |a|.
inline pair16 grow_two_sum(pair16 xy, bf16 a) {
    pair16 uv = two_sum(xy.hi, a);
    return two_sum(uv.hi, op_add(xy.lo, uv.lo));
}

struct edq_sums { double dot, sumsq; uint64_t lost; };

// Is the effective update (theta' + dtheta') - (theta + dtheta) of Eq. 2 zero?  A yes/no decision taken
// by floating point: it is evaluated in single precision, differences first, the precision in which the
// device forms the same quantity, so that both sides decide alike on every input.  For normalised
// expansions (|lo| <= ulp(hi)/2, which Grow maintains) the single-precision result is zero exactly when
// the real number is: each difference of two bfloat16 values is either exact in single precision or so
// large that the other difference cannot cancel it, and an IEEE addition of two non-zero numbers gives
// zero only when they are opposite.  tests/test_oracle_step.py checks this against exact rationals.
inline bool value_unchanged(bf16 hi_old, bf16 lo_old, bf16 hi_new, bf16 lo_new, bool pair) {
    const float move_hi = static_cast<float>(widen(hi_new)) - static_cast<float>(widen(hi_old));
    if (!pair) return move_hi == 0.0f;
    const float move_lo = static_cast<float>(widen(lo_new)) - static_cast<float>(widen(lo_old));
    return move_hi + move_lo == 0.0f;
}

// One parameter, one step of Algorithm 2 (lines 8-13), in the printed order.
// Returns the bfloat16 update (line 12) and accumulates the EDQ sums
// (Eq. 2 and Eq. 3) in double.
inline void step_one(bf16& th, bf16* dth, bf16& m, bf16& v, bf16* dv, bf16 g,
                     const scalars& s, int strategy, uint32_t flags,
                     bf16* delta_out, edq_sums& acc) {
    // line 8: first moment
    m = op_add(op_mul(s.b1, m), op_mul(s.c1, g));
    // line 9: increment (1-beta2) * g^2, g^2 first (reading)
    const bf16 tv = op_mul(s.c2, op_mul(g, g));
    if (strategy == STRAT_PLUS) {
        // line 9, highlighted form: Grow(Mul((b2h,b2l),(v,dv)), tv)
        pair16 decayed = mul(pair16{s.b2h, s.b2l}, pair16{v, *dv});
        pair16 nv = grow(decayed, tv);
        v = nv.hi;
        *dv = nv.lo;
    } else {
        v = op_add(op_mul(s.b2, v), tv);
    }
    // lines 10-11: bias corrections; first component of v only (reading)
    const bf16 mhat = op_div(m, s.bc1);
    const bf16 vhat = op_div(v, s.bc2);
    // line 12: epsilon outside the root as in AdamW; the literal printed form
    // (inside) is selectable (reading)
    bf16 den;
    if (flags & FLAG_EPS_INSIDE_SQRT) den = op_sqrt(op_add(vhat, s.eps));
    else den = op_add(op_sqrt(vhat), s.eps);
    const bf16 r = op_div(mhat, den);
    const bf16 w = op_mul(s.lam, th);          // decay uses the first component of theta (reading)
    // Appendix D, weight decay: either summed into the update (default, "the latter option"), or
    // applied to the parameter by an addition of its own (flag): d = -a (*) (lam (*) theta).
    const bool split_decay = (flags & FLAG_DECAY_BY_GROW) != 0;
    const bf16 decay = op_mul(op_neg(s.a), w);
    const bf16 delta = split_decay ? op_mul(op_neg(s.a), r) : op_mul(op_neg(s.a), op_add(r, w));
    // line 13
    const bf16 th_old = th;
    const bf16 dth_old = dth ? *dth : 0;
    auto add_to_parameter = [&](bf16 upd) {
        if (strategy == STRAT_BF16) {
            th = op_add(th, upd);              // Eq. 1
        } else {
            pair16 nt = (flags & FLAG_TWOSUM_GROW) ? grow_two_sum(pair16{th, *dth}, upd) : grow(pair16{th, *dth}, upd);
            th = nt.hi;
            *dth = nt.lo;
        }
    };
    if (strategy == STRAT_KAHAN) {
        // Appendix B, Kahan summation: the compensation c (stored where dtheta would be) is added to the
        // update, and c <- F(update (-) F(theta_t (-) theta_{t-1})) is kept for the next step
        const bf16 comp = op_add(delta, *dth);
        th = op_add(th_old, comp);
        *dth = op_sub(comp, op_sub(th, th_old));
    } else {
        if (split_decay) add_to_parameter(decay);
        add_to_parameter(delta);
    }
    // Eq. 2 generalised to an expansion: effective update = (theta'+dtheta') - (theta+dtheta).  For Kahan
    // the parameter is theta alone (Eq. 2 as printed); c is bookkeeping, not part of the value.
    const bool pair_value = dth && strategy != STRAT_KAHAN;
    const double eff = (widen(th) - widen(th_old)) + (pair_value ? (widen(*dth) - widen(dth_old)) : 0.0);
    const double d = widen(delta) + (split_decay ? widen(decay) : 0.0);      // intended update
    acc.dot += d * eff;
    acc.sumsq += d * d;
    // lost arithmetic (Def. 3.2; "not updated", Figure 3 left): an update was intended and the parameter
    // did not move, i.e. the effective update of Eq. 2 is zero.  For an expansion the parameter is the
    // value theta + dtheta: a Grow that re-splits the same value over other components has not updated it.
    if (d != 0.0 && value_unchanged(th_old, dth_old, th, pair_value ? *dth : 0, pair_value)) acc.lost += 1;
    if (delta_out) *delta_out = delta;
}

}  // namespace

extern "C" {

// ---- format ----------------------------------------------------------------
uint16_t oracle_round_to_bf16(double x) { return round_to_bf16(x); }
double oracle_bf16_to_double(uint16_t h) { return widen(h); }

void oracle_round_array(const double* x, uint16_t* out, uint64_t n) {
    for (uint64_t i = 0; i < n; ++i) out[i] = round_to_bf16(x[i]);
}
void oracle_widen_array(const uint16_t* h, double* out, uint64_t n) {
    for (uint64_t i = 0; i < n; ++i) out[i] = widen(h[i]);
}

// ---- single rounded operations, elementwise --------------------------------
// op: 0 add, 1 sub, 2 mul, 3 div, 4 sqrt(a), 5 fma(a,b,c)
void oracle_binary_op(int op, const uint16_t* a, const uint16_t* b, const uint16_t* c,
                      uint16_t* out, uint64_t n) {
    for (uint64_t i = 0; i < n; ++i) {
        switch (op) {
            case 0: out[i] = op_add(a[i], b[i]); break;
            case 1: out[i] = op_sub(a[i], b[i]); break;
            case 2: out[i] = op_mul(a[i], b[i]); break;
            case 3: out[i] = op_div(a[i], b[i]); break;
            case 4: out[i] = op_sqrt(a[i]); break;
            case 5: out[i] = op_fma(a[i], b[i], c[i]); break;
            default: out[i] = 0x7FC0u;
        }
    }
}

// ---- MCF primitives, elementwise -------------------------------------------
void oracle_fast_two_sum(const uint16_t* a, const uint16_t* b, uint16_t* hi, uint16_t* lo, uint64_t n) {
    for (uint64_t i = 0; i < n; ++i) { pair16 r = fast_two_sum(a[i], b[i]); hi[i] = r.hi; lo[i] = r.lo; }
}
void oracle_two_sum(const uint16_t* a, const uint16_t* b, uint16_t* hi, uint16_t* lo, uint64_t n) {
    for (uint64_t i = 0; i < n; ++i) { pair16 r = two_sum(a[i], b[i]); hi[i] = r.hi; lo[i] = r.lo; }
}
void oracle_two_prod(const uint16_t* a, const uint16_t* b, uint16_t* hi, uint16_t* lo, uint64_t n) {
    for (uint64_t i = 0; i < n; ++i) { pair16 r = two_prod_fma(a[i], b[i]); hi[i] = r.hi; lo[i] = r.lo; }
}
void oracle_two_prod_dekker(const uint16_t* a, const uint16_t* b, uint16_t* hi, uint16_t* lo, uint64_t n) {
    for (uint64_t i = 0; i < n; ++i) { pair16 r = two_prod_dekker(a[i], b[i]); hi[i] = r.hi; lo[i] = r.lo; }
}
void oracle_split(const uint16_t* a, uint16_t* hi, uint16_t* lo, uint64_t n) {
    for (uint64_t i = 0; i < n; ++i) { pair16 r = split(a[i]); hi[i] = r.hi; lo[i] = r.lo; }
}
void oracle_grow(const uint16_t* x, const uint16_t* y, const uint16_t* a, uint16_t* u, uint16_t* v, uint64_t n) {
    for (uint64_t i = 0; i < n; ++i) { pair16 r = grow(pair16{x[i], y[i]}, a[i]); u[i] = r.hi; v[i] = r.lo; }
}
void oracle_scaling(const uint16_t* v, const uint16_t* a1, const uint16_t* a2, uint16_t* x, uint16_t* e, uint64_t n) {
    for (uint64_t i = 0; i < n; ++i) { pair16 r = scaling(v[i], pair16{a1[i], a2[i]}); x[i] = r.hi; e[i] = r.lo; }
}
void oracle_mul(const uint16_t* a1, const uint16_t* a2, const uint16_t* b1, const uint16_t* b2,
                uint16_t* x, uint16_t* e, uint64_t n) {
    for (uint64_t i = 0; i < n; ++i) {
        pair16 r = mul(pair16{a1[i], a2[i]}, pair16{b1[i], b2[i]});
        x[i] = r.hi; e[i] = r.lo;
    }
}
void oracle_renormalize(const uint16_t* hi_in, const uint16_t* lo_in, uint16_t* hi, uint16_t* lo, uint64_t n) {
    for (uint64_t i = 0; i < n; ++i) { pair16 r = renormalize(pair16{hi_in[i], lo_in[i]}); hi[i] = r.hi; lo[i] = r.lo; }
}

// ---- scalars -----------------------------------------------------------------
// out[11] = b1, c1, b2, c2, b2h, b2l, bc1, bc2, a, lam, eps
void oracle_derive_scalars(double lr, double beta1, double beta2, double eps, double wd,
                           uint64_t step, uint16_t* out) {
    const scalars s = derive_scalars(lr, beta1, beta2, eps, wd, step);
    out[0] = s.b1; out[1] = s.c1; out[2] = s.b2; out[3] = s.c2; out[4] = s.b2h; out[5] = s.b2l;
    out[6] = s.bc1; out[7] = s.bc2; out[8] = s.a; out[9] = s.lam; out[10] = s.eps;
}

// ---- the step ------------------------------------------------------------------
// Algorithm 2, one call = one step t over n parameters, in place.
// x_lo may be NULL for strategy 0; v_lo may be NULL unless strategy 2.
// delta_out (optional, n entries) receives the bfloat16 update of line 12.
// sums_out[4] = {dot, sumsq, edq, lost} with EDQ = dot / sqrt(sumsq) (Eq. 3),
// 0 when the update norm is 0.  threads <= 1: one pass in index order.
// threads > 1: contiguous index ranges, each summed in index order, range
// sums added in range order.
void oracle_adamw_step(uint16_t* x_hi, uint16_t* x_lo, uint16_t* m, uint16_t* v_hi, uint16_t* v_lo,
                       const uint16_t* grad, uint64_t n,
                       double lr, double beta1, double beta2, double eps, double wd, uint32_t flags,
                       uint64_t step, int strategy, uint16_t* delta_out, double* sums_out, int threads) {
    const scalars s = derive_scalars(lr, beta1, beta2, eps, wd, step);
    if (threads < 1) threads = 1;
    std::vector<edq_sums> part(static_cast<size_t>(threads), edq_sums{0.0, 0.0, 0});
#ifdef _OPENMP
#pragma omp parallel for num_threads(threads) schedule(static, 1)
#endif
    for (int r = 0; r < threads; ++r) {
        const uint64_t lo = n / threads * r + std::min<uint64_t>(r, n % threads);
        const uint64_t hi = lo + n / threads + (static_cast<uint64_t>(r) < n % threads ? 1 : 0);
        edq_sums acc{0.0, 0.0, 0};
        for (uint64_t i = lo; i < hi; ++i) {
            step_one(x_hi[i], strategy != STRAT_BF16 ? &x_lo[i] : nullptr, m[i], v_hi[i],
                     strategy == STRAT_PLUS ? &v_lo[i] : nullptr, grad[i], s, strategy, flags,
                     delta_out ? &delta_out[i] : nullptr, acc);
        }
        part[static_cast<size_t>(r)] = acc;
    }
    edq_sums tot{0.0, 0.0, 0};
    for (const edq_sums& p : part) { tot.dot += p.dot; tot.sumsq += p.sumsq; tot.lost += p.lost; }
    if (sums_out) {
        sums_out[0] = tot.dot;
        sums_out[1] = tot.sumsq;
        sums_out[2] = tot.sumsq > 0.0 ? tot.dot / std::sqrt(tot.sumsq) : 0.0;
        sums_out[3] = static_cast<double>(tot.lost);
    }
}

// Eq. 2-3 on stored arrays: old/new expansions and the intended update.
// old_lo/new_lo may be NULL (plain bfloat16 parameter).
void oracle_edq(const uint16_t* old_hi, const uint16_t* old_lo, const uint16_t* new_hi,
                const uint16_t* new_lo, const uint16_t* delta, uint64_t n, double* sums_out) {
    edq_sums tot{0.0, 0.0, 0};
    for (uint64_t i = 0; i < n; ++i) {
        double eff = widen(new_hi[i]) - widen(old_hi[i]);
        if (old_lo && new_lo) eff += widen(new_lo[i]) - widen(old_lo[i]);
        const double d = widen(delta[i]);
        tot.dot += d * eff;
        tot.sumsq += d * d;
        const bool pair = old_lo && new_lo;
        if (d != 0.0 && value_unchanged(old_hi[i], pair ? old_lo[i] : 0, new_hi[i], pair ? new_lo[i] : 0, pair)) tot.lost += 1;
    }
    sums_out[0] = tot.dot;
    sums_out[1] = tot.sumsq;
    sums_out[2] = tot.sumsq > 0.0 ? tot.dot / std::sqrt(tot.sumsq) : 0.0;
    sums_out[3] = static_cast<double>(tot.lost);
}

// AdamW of Loshchilov & Hutter with the same formulas as Algorithm 2, all in
// double, no rounding to bfloat16 anywhere: the "what the step approximates"
// reference.  Returns the update in delta_out if given.
void oracle_adamw_fp64(double* theta, double* m, double* v, const double* grad, uint64_t n,
                       double lr, double beta1, double beta2, double eps, double wd,
                       uint32_t flags, uint64_t step, double* delta_out) {
    const double bc1 = 1.0 - std::pow(beta1, static_cast<double>(step));
    const double bc2 = 1.0 - std::pow(beta2, static_cast<double>(step));
    for (uint64_t i = 0; i < n; ++i) {
        m[i] = beta1 * m[i] + (1.0 - beta1) * grad[i];
        v[i] = beta2 * v[i] + (1.0 - beta2) * grad[i] * grad[i];
        const double mhat = m[i] / bc1, vhat = v[i] / bc2;
        const double den = (flags & FLAG_EPS_INSIDE_SQRT) ? std::sqrt(vhat + eps) : std::sqrt(vhat) + eps;
        const double d = -lr * (mhat / den + wd * theta[i]);
        theta[i] += d;
        if (delta_out) delta_out[i] = d;
    }
}

// ---- comparator: option D of Table 2 (bfloat16 parameter and gradient, float optimizer states,
// float master weights) and D^-MW (Section 5.1: the same without master weights) -----------------
// Standard mixed-precision AdamW: every operation below is one IEEE single-precision operation
// (this file is compiled with contraction off), scalars are evaluated in double and cast to float
// once (Appendix D, scalar rule).  master == NULL selects D^-MW: the update is added to the
// bfloat16 parameter widened to float and the sum is rounded back to bfloat16.
// EDQ (Eq. 2-3): intended update = the float update; effective update = change of the stored
// parameter (the master weight for D, the bfloat16 parameter for D^-MW), summed in double.
void oracle_adamw_fp32_step(uint16_t* theta, float* master, float* m, float* v, const uint16_t* grad, uint64_t n,
                            double lr, double beta1, double beta2, double eps, double wd, uint32_t flags,
                            uint64_t step, double* sums_out) {
    const float b1 = static_cast<float>(beta1), c1 = static_cast<float>(1.0 - beta1);
    const float b2 = static_cast<float>(beta2), c2 = static_cast<float>(1.0 - beta2);
    const float bc1 = static_cast<float>(1.0 - std::pow(beta1, static_cast<double>(step)));
    const float bc2 = static_cast<float>(1.0 - std::pow(beta2, static_cast<double>(step)));
    const float neg_a = -static_cast<float>(lr), lam = static_cast<float>(wd), epsf = static_cast<float>(eps);
    edq_sums tot{0.0, 0.0, 0};
    for (uint64_t i = 0; i < n; ++i) {
        const float g = static_cast<float>(widen(grad[i]));
        const float m_new = b1 * m[i] + c1 * g;
        const float gg = g * g;
        const float v_new = b2 * v[i] + c2 * gg;
        m[i] = m_new;
        v[i] = v_new;
        const float mhat = m_new / bc1;
        const float vhat = v_new / bc2;
        const float den = (flags & FLAG_EPS_INSIDE_SQRT) ? std::sqrt(vhat + epsf) : std::sqrt(vhat) + epsf;
        const float w_old = master ? master[i] : static_cast<float>(widen(theta[i]));
        const float r = mhat / den;
        const float decay = lam * w_old;
        const float u = r + decay;
        const float delta = neg_a * u;
        const float w_new = w_old + delta;
        const uint16_t theta_new = round_to_bf16(static_cast<double>(w_new));
        double eff;
        bool unchanged;
        if (master) {
            master[i] = w_new;
            eff = static_cast<double>(w_new) - static_cast<double>(w_old);
            unchanged = (w_new == w_old);
        } else {
            eff = widen(theta_new) - widen(theta[i]);
            unchanged = (widen(theta_new) == widen(theta[i]));
        }
        theta[i] = theta_new;
        const double d = static_cast<double>(delta);
        tot.dot += d * eff;
        tot.sumsq += d * d;
        if (d != 0.0 && unchanged) tot.lost += 1;
    }
    if (sums_out) {
        sums_out[0] = tot.dot;
        sums_out[1] = tot.sumsq;
        sums_out[2] = tot.sumsq > 0.0 ? tot.dot / std::sqrt(tot.sumsq) : 0.0;
        sums_out[3] = static_cast<double>(tot.lost);
    }
}

// ---- variant: float arithmetic in registers on the Collage-plus storage -------------------------
// Not in the paper (its Algorithm 2 is strict bfloat16); a measuring stick for what the strict
// arithmetic costs at equal memory traffic.  Storage is option C's: (theta, dtheta), m, (v, dv) in
// bfloat16.  Each step widens to float (theta + dtheta and v + dv by one float addition), runs
// AdamW exactly as the option-D comparator does (IEEE single operations, float scalars), and
// splits the results back: hi = RN_bf16(x), lo = RN_bf16(x - hi).
void oracle_adamw_fp32_register_step(uint16_t* x_hi, uint16_t* x_lo, uint16_t* m, uint16_t* v_hi, uint16_t* v_lo,
                                     const uint16_t* grad, uint64_t n, double lr, double beta1, double beta2,
                                     double eps, double wd, uint32_t flags, uint64_t step, double* sums_out) {
    const float b1 = static_cast<float>(beta1), c1 = static_cast<float>(1.0 - beta1);
    const float b2 = static_cast<float>(beta2), c2 = static_cast<float>(1.0 - beta2);
    const float bc1 = static_cast<float>(1.0 - std::pow(beta1, static_cast<double>(step)));
    const float bc2 = static_cast<float>(1.0 - std::pow(beta2, static_cast<double>(step)));
    const float neg_a = -static_cast<float>(lr), lam = static_cast<float>(wd), epsf = static_cast<float>(eps);
    auto f = [](uint16_t h) { return static_cast<float>(widen(h)); };
    edq_sums tot{0.0, 0.0, 0};
    for (uint64_t i = 0; i < n; ++i) {
        const float g = f(grad[i]);
        const float x = f(x_hi[i]) + f(x_lo[i]);
        const float vv = f(v_hi[i]) + f(v_lo[i]);
        const float m_new = b1 * f(m[i]) + c1 * g;
        const float gg = g * g;
        const float v_new = b2 * vv + c2 * gg;
        const float mhat = m_new / bc1;
        const float vhat = v_new / bc2;
        const float den = (flags & FLAG_EPS_INSIDE_SQRT) ? std::sqrt(vhat + epsf) : std::sqrt(vhat) + epsf;
        const float r = mhat / den;
        const float decay = lam * x;
        const float u = r + decay;
        const float delta = neg_a * u;
        const float x_new = x + delta;
        const uint16_t th = round_to_bf16(static_cast<double>(x_new));
        const uint16_t dth = round_to_bf16(static_cast<double>(x_new - f(th)));
        const uint16_t vh = round_to_bf16(static_cast<double>(v_new));
        const uint16_t vl = round_to_bf16(static_cast<double>(v_new - f(vh)));
        const double eff = (widen(th) - widen(x_hi[i])) + (widen(dth) - widen(x_lo[i]));
        const bool unchanged = value_unchanged(x_hi[i], x_lo[i], th, dth, true);
        x_hi[i] = th;
        x_lo[i] = dth;
        m[i] = round_to_bf16(static_cast<double>(m_new));
        v_hi[i] = vh;
        v_lo[i] = vl;
        const double d = static_cast<double>(delta);
        tot.dot += d * eff;
        tot.sumsq += d * d;
        if (d != 0.0 && unchanged) tot.lost += 1;
    }
    if (sums_out) {
        sums_out[0] = tot.dot;
        sums_out[1] = tot.sumsq;
        sums_out[2] = tot.sumsq > 0.0 ? tot.dot / std::sqrt(tot.sumsq) : 0.0;
        sums_out[3] = static_cast<double>(tot.lost);
    }
}

int oracle_max_threads(void) {
#ifdef _OPENMP
    return omp_get_max_threads();
#else
    return 1;
#endif
}

}  // extern "C"
