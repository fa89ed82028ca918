// Device-side bfloat16 arithmetic and the multi-component-float (MCF) algorithms of the paper,
// two elements at a time.
//
// A `bf2` is a 32-bit register holding two bfloat16 values.  Every function below applies the
// same operation to both halves.  The arithmetic model is Section 3.1's F^BF16(a op b): each
// operator rounds its exact result once to bfloat16, nearest-even.
//
//   add/sub/mul/fma : the native packed instructions add/sub/mul/fma.rn.bf16x2 (sm_90+), one
//                     rounding, subnormals kept, written as inline PTX so that nothing can be
//                     contracted, re-associated or flushed by the compiler.
//   div, sqrt       : no bfloat16 instruction exists.  Operands are widened to float (exact) and
//                     a float result q is formed that rounds (cvt.rn.bf16x2.f32) to the same
//                     bfloat16 as the exact quotient / root:
//                       * IEEE route: div.rn.f32 / sqrt.rn.f32.  24 bits >= 2*8+2, so the second
//                         rounding is innocuous.
//                       * fast route (default): a * rcp.approx.ftz(b), a * (1/b rounded to float on
//                         the host) for the two scalar divisors, and sqrt.approx.ftz.f32.  Their relative
//                         error is <= 2^-22, while the exact quotient of two 8-bit significands is
//                         never an exact tie and never closer than 2^-17 (relative) to a rounding
//                         boundary, and a square root never closer than 2^-19; so the approximation
//                         and the exact value round alike.  The argument needs a normal-range
//                         result: anything else (tiny, huge, Inf, NaN) takes the IEEE route; 0/b is answered directly.
//                         collage_selftest() compares the two routes over every operand pair.
//
// This file is compiled only into the CUDA library; it shares nothing with the CPU oracle.
#pragma once
#include <cstdint>
#include <cuda_runtime.h>

namespace collage {

typedef uint32_t bf2;

// ------------------------------------------------------------ rounded ops ---

__device__ __forceinline__ bf2 add2(bf2 a, bf2 b) {
    bf2 d;
    asm("add.rn.bf16x2 %0, %1, %2;" : "=r"(d) : "r"(a), "r"(b));
    return d;
}
__device__ __forceinline__ bf2 sub2(bf2 a, bf2 b) {
    bf2 d;
    asm("sub.rn.bf16x2 %0, %1, %2;" : "=r"(d) : "r"(a), "r"(b));
    return d;
}
__device__ __forceinline__ bf2 mul2(bf2 a, bf2 b) {
    bf2 d;
    asm("mul.rn.bf16x2 %0, %1, %2;" : "=r"(d) : "r"(a), "r"(b));
    return d;
}
__device__ __forceinline__ bf2 fma2(bf2 a, bf2 b, bf2 c) {
    bf2 d;
    asm("fma.rn.bf16x2 %0, %1, %2, %3;" : "=r"(d) : "r"(a), "r"(b), "r"(c));
    return d;
}
__device__ __forceinline__ bf2 neg2(bf2 a) { return a ^ 0x80008000u; }

// widen the low / high half to float (exact)
__device__ __forceinline__ float lo_f32(bf2 p) { return __uint_as_float(p << 16); }
__device__ __forceinline__ float hi_f32(bf2 p) { return __uint_as_float(p & 0xFFFF0000u); }

// round two floats to bfloat16 (nearest-even) and pack: `hi` to the upper half
__device__ __forceinline__ bf2 pack_rn(float hi, float lo) {
    bf2 d;
    asm("cvt.rn.bf16x2.f32 %0, %1, %2;" : "=r"(d) : "f"(hi), "f"(lo));
    return d;
}

// two floats as one 64-bit register pair for the packed f32x2 instructions of sm_100
typedef unsigned long long f32x2;
__device__ __forceinline__ f32x2 widen2(bf2 p) {      // {low half, high half} as floats (exact)
    f32x2 d;
    asm("mov.b64 %0, {%1, %2};" : "=l"(d) : "r"(p << 16), "r"(p & 0xFFFF0000u));
    return d;
}
__device__ __forceinline__ f32x2 splat2(float x) {
    f32x2 d;
    asm("mov.b64 %0, {%1, %1};" : "=l"(d) : "f"(x));
    return d;
}
__device__ __forceinline__ f32x2 mul_f32x2(f32x2 a, f32x2 b) {
    f32x2 d;
    asm("mul.rn.f32x2 %0, %1, %2;" : "=l"(d) : "l"(a), "l"(b));
    return d;
}
__device__ __forceinline__ f32x2 add_f32x2(f32x2 a, f32x2 b) {
    f32x2 d;
    asm("add.rn.f32x2 %0, %1, %2;" : "=l"(d) : "l"(a), "l"(b));
    return d;
}
__device__ __forceinline__ f32x2 sub_f32x2(f32x2 a, f32x2 b) {
    f32x2 d;
    asm("sub.rn.f32x2 %0, %1, %2;" : "=l"(d) : "l"(a), "l"(b));
    return d;
}
__device__ __forceinline__ f32x2 fma_f32x2(f32x2 a, f32x2 b, f32x2 c) {
    f32x2 d;
    asm("fma.rn.f32x2 %0, %1, %2, %3;" : "=l"(d) : "l"(a), "l"(b), "l"(c));
    return d;
}
__device__ __forceinline__ float lo_of(f32x2 v) { return __uint_as_float(static_cast<uint32_t>(v)); }
__device__ __forceinline__ float hi_of(f32x2 v) { return __uint_as_float(static_cast<uint32_t>(v >> 32)); }
// round both floats to bfloat16 and pack (low float to the low half)
__device__ __forceinline__ bf2 pack_rn2(f32x2 v) { return pack_rn(hi_of(v), lo_of(v)); }

// IEEE routes (also the fall-back of the fast routes)
__device__ __forceinline__ bf2 div2_ieee(bf2 a, bf2 b) {
    return pack_rn(__fdiv_rn(hi_f32(a), hi_f32(b)), __fdiv_rn(lo_f32(a), lo_f32(b)));
}
__device__ __forceinline__ bf2 sqrt2_ieee(bf2 a) {
    return pack_rn(__fsqrt_rn(hi_f32(a)), __fsqrt_rn(lo_f32(a)));
}
static __device__ __noinline__ float div_ieee_call(float a, float b) { return __fdiv_rn(a, b); }
static __device__ __noinline__ float sqrt_ieee_call(float a) { return __fsqrt_rn(a); }

// Quotient for operands the fast route does not cover.  A zero numerator over a normal finite
// denominator is common (parameters that never received a gradient) and is answered directly:
// a zero with the sign of the quotient.  Everything else goes to div.rn.f32.
__device__ __forceinline__ float div_out_of_range(float a, float b) {
    if (a == 0.0f && fabsf(b) >= 0x1p-126f && fabsf(b) < __uint_as_float(0x7F800000u))
        return __uint_as_float((__float_as_uint(a) ^ __float_as_uint(b)) & 0x80000000u);
    return div_ieee_call(a, b);
}

// single MUFU approximations; .ftz flushes subnormal inputs and outputs, which the callers below
// either exclude or detect
__device__ __forceinline__ float rcp_ftz(float b) {
    float r;
    asm("rcp.approx.ftz.f32 %0, %1;" : "=f"(r) : "f"(b));
    return r;
}
__device__ __forceinline__ float sqrt_ftz(float a) {
    float r;
    asm("sqrt.approx.ftz.f32 %0, %1;" : "=f"(r) : "f"(a));
    return r;
}

// q is trusted only if it is a normal number with room to spare on both sides.  A subnormal
// denominator is flushed by rcp.approx.ftz (q = Inf or NaN), a denominator above 2^126 gives a
// flushed reciprocal (q = 0): both fail the test, as does a NaN.
__device__ __forceinline__ bool quotient_in_fast_range(float q) {
    return fabsf(q) >= 0x1p-125f && fabsf(q) < 0x1p127f;
}

// a (/) b, both halves, any operands
__device__ __forceinline__ bf2 div2(bf2 a, bf2 b) {
#ifdef COLLAGE_IEEE_DIV_SQRT
    return div2_ieee(a, b);
#else
    const float a0 = lo_f32(a), a1 = hi_f32(a), b0 = lo_f32(b), b1 = hi_f32(b);
    float q0 = __fmul_rn(a0, rcp_ftz(b0));
    float q1 = __fmul_rn(a1, rcp_ftz(b1));
    if (!(quotient_in_fast_range(q0) && quotient_in_fast_range(q1))) {
        if (!quotient_in_fast_range(q0)) q0 = div_out_of_range(a0, b0);
        if (!quotient_in_fast_range(q1)) q1 = div_out_of_range(a1, b1);
    }
    return pack_rn(q1, q0);
#endif
}

// a (/) s for a scalar 2^-100 <= s <= 1 whose reciprocal r was rounded to float on the host.
// No range test is needed: |a*r| >= |a|, so a quotient can only be subnormal when a is, and then
// both the float product and the exact quotient sit on grids (2^-149 and 1/(256*2^134)) that keep
// them on the same side of every rounding boundary; a divisor <= 1 admits no exact tie; an
// overflowing product is the overflowing quotient; zeros, Inf and NaN pass through unchanged.
__device__ __forceinline__ bf2 div2_by_scalar(bf2 a, float r) { return pack_rn2(mul_f32x2(widen2(a), splat2(r))); }

// the same for any scalar: falls back to IEEE division when the host did not vouch (r is NaN)
__device__ __forceinline__ bf2 div2_scalar(bf2 a, float s, float r) {
#ifdef COLLAGE_IEEE_DIV_SQRT
    return pack_rn(__fdiv_rn(hi_f32(a), s), __fdiv_rn(lo_f32(a), s));
#else
    if (r == r) return div2_by_scalar(a, r);
    return pack_rn(__fdiv_rn(hi_f32(a), s), __fdiv_rn(lo_f32(a), s));
#endif
}

// sqrt(a), both halves, any operand: the approximation flushes subnormal inputs, which go to sqrt.rn
__device__ __forceinline__ bf2 sqrt2(bf2 a) {
#ifdef COLLAGE_IEEE_DIV_SQRT
    return sqrt2_ieee(a);
#else
    const float a0 = lo_f32(a), a1 = hi_f32(a);
    float s0 = sqrt_ftz(a0), s1 = sqrt_ftz(a1);
    if ((a0 != 0.0f && fabsf(a0) < 0x1p-126f) || (a1 != 0.0f && fabsf(a1) < 0x1p-126f)) {
        s0 = sqrt_ieee_call(a0);
        s1 = sqrt_ieee_call(a1);
    }
    return pack_rn(s1, s0);
#endif
}
// all-ones in each half of the result where that half of a is < b (false for NaN)
__device__ __forceinline__ uint32_t less_than2(bf2 a, bf2 b) {
    uint32_t d;
    asm("set.lt.u32.bf16x2 %0, %1, %2;" : "=r"(d) : "r"(a), "r"(b));
    return d;
}
// ---- deferred forms: no branch; a lane the fast route cannot answer sets bits in `suspect`, and
// the caller recomputes the whole vector by the careful routes when any bit is set ---------------
__device__ __forceinline__ uint32_t less_equal2(bf2 a, bf2 b) {
    uint32_t d;
    asm("set.le.u32.bf16x2 %0, %1, %2;" : "=r"(d) : "r"(a), "r"(b));
    return d;
}
// all-ones where the halves differ or either is NaN
__device__ __forceinline__ uint32_t differs2(bf2 a, bf2 b) {
    uint32_t d;
    asm("set.neu.u32.bf16x2 %0, %1, %2;" : "=r"(d) : "r"(a), "r"(b));
    return d;
}
__device__ __forceinline__ uint32_t equal2(bf2 a, bf2 b) {
    uint32_t d;
    asm("set.eq.u32.bf16x2 %0, %1, %2;" : "=r"(d) : "r"(a), "r"(b));
    return d;
}
// a (/) b where the caller guarantees that b is NaN, Inf, or a normal number in [2^-126, 2^126]:
// the reciprocal is then accurate and an overflowing quotient is correctly Inf.  The rounded
// quotient is trusted unless its magnitude is at most 2^-125 (the float product may then have
// been subnormal or tied) while the numerator is not zero; a zero numerator gives the correctly
// signed zero (or NaN for a NaN divisor) by the product alone, and a NaN product is a NaN quotient
// for every admitted divisor.
__device__ __forceinline__ bf2 div2_normal_divisor_deferred(bf2 a, bf2 b, uint32_t& suspect) {
#ifdef COLLAGE_IEEE_DIV_SQRT
    return div2_ieee(a, b);
#else
    const bf2 q = pack_rn(__fmul_rn(hi_f32(a), rcp_ftz(hi_f32(b))), __fmul_rn(lo_f32(a), rcp_ftz(lo_f32(b))));
    suspect |= less_equal2(q & 0x7FFF7FFFu, 0x01000100u) & ~equal2(a, 0u);   // 0x0100 = 2^-125
    return q;
#endif
}
// sqrt(a) where the caller accepts +0 for a positive subnormal input (true root < 2^-63: the
// approximation flushes it).  A negative lane (NaN by IEEE, but -0 from the flushing approximation
// when subnormal) marks the vector.
__device__ __forceinline__ bf2 sqrt2_flushing_deferred(bf2 a, uint32_t& suspect) {
#ifdef COLLAGE_IEEE_DIV_SQRT
    return sqrt2_ieee(a);
#else
    suspect |= less_than2(a, 0u);
    return pack_rn(sqrt_ftz(hi_f32(a)), sqrt_ftz(lo_f32(a)));
#endif
}

// --------------------------------------------------------- MCF algorithms ---

struct bf2pair {
    bf2 hi, lo;
};

// Theorem 4.1 (Fast2Sum), applied without sorting
__device__ __forceinline__ bf2pair fast_two_sum2(bf2 a, bf2 b) {
    bf2pair r;
    r.hi = add2(a, b);
    r.lo = sub2(b, sub2(r.hi, a));
    return r;
}

// Algorithm TwoSum (Appendix C)
__device__ __forceinline__ bf2pair two_sum2(bf2 a, bf2 b) {
    bf2pair r;
    r.hi = add2(a, b);
    const bf2 bv = sub2(r.hi, a);
    const bf2 av = sub2(r.hi, bv);
    const bf2 br = sub2(b, bv);
    const bf2 ar = sub2(a, av);
    r.lo = add2(ar, br);
    return r;
}

// Algorithm TwoProdFMA (Appendix C)
__device__ __forceinline__ bf2pair two_prod2(bf2 a, bf2 b) {
    bf2pair r;
    r.hi = mul2(a, b);
    r.lo = fma2(a, b, neg2(r.hi));
    return r;
}

// Algorithm 1 (Grow): expansion (x, y) plus float a
__device__ __forceinline__ bf2pair grow2(bf2 x, bf2 y, bf2 a) {
    const bf2pair s = fast_two_sum2(x, a);
    return fast_two_sum2(s.hi, add2(y, s.lo));
}

// Grow with TwoSum in place of Fast2Sum (Appendix C): error-free for any ordering of |x| and |a|
__device__ __forceinline__ bf2pair grow_two_sum2(bf2 x, bf2 y, bf2 a) {
    const bf2pair s = two_sum2(x, a);
    return two_sum2(s.hi, add2(y, s.lo));
}

// Algorithm Scaling: float v times expansion (a1, a2)
__device__ __forceinline__ bf2pair scaling2(bf2 v, bf2 a1, bf2 a2) {
    const bf2pair p = two_prod2(a1, v);
    const bf2 e = add2(mul2(a2, v), p.lo);
    return fast_two_sum2(p.hi, e);
}

// Algorithm Mul: expansion (a1, a2) times expansion (b1, b2)
__device__ __forceinline__ bf2pair mcf_mul2(bf2 a1, bf2 a2, bf2 b1, bf2 b2) {
    const bf2pair p = two_prod2(a1, b1);
    const bf2 cross = add2(mul2(a1, b2), mul2(a2, b1));
    const bf2 e = add2(p.lo, cross);
    return fast_two_sum2(p.hi, e);
}

// ------------------------------------------------------------ AdamW step ---

// float scalars of the register variant (cast from double once, like the option-D comparator's)
struct FloatScalars {
    float b1, c1, b2, c2, bc1, bc2, neg_a, lam, eps;
};

// bfloat16 scalars of one step, each duplicated into both halves of a bf2 (Algorithm 2 line 1).
struct StepScalars {
    bf2 b1, c1;        // RN(beta1), RN(1-beta1)
    bf2 b2, c2;        // RN(beta2), RN(1-beta2)
    bf2 b2h, b2l;      // beta2 as a length-2 expansion (Table 1)
    float bc1, bc2;    // RN(1-beta1^t), RN(1-beta2^t) widened to float
    float rbc1, rbc2;  // their reciprocals rounded to float (NaN: use the IEEE route)
    bf2 neg_a;         // -RN(lr)
    bf2 lam;           // RN(weight_decay)
    bf2 eps;           // RN(eps)
    uint32_t flags;    // bit 0: epsilon under the root; bit 1: TwoSum Grow; bit 2: decay by its own addition
    uint32_t fast;     // host-checked: 2^-100 <= bc1, bc2 <= 1 and 2^-54 <= eps <= 2^60
    FloatScalars f;    // only read by the register variant (strategy 4)
};

struct ElemState {
    bf2 th, dth, m, v, dv;
};

// which arrays a strategy stores: 0 = A, 1 = B, 2 = C, 3 = BF16-Kahan, 4 = float arithmetic in
// registers on option C's storage
__host__ __device__ constexpr bool stores_x_lo(int strategy) { return strategy >= 1; }
__host__ __device__ constexpr bool stores_v_lo(int strategy) { return strategy == 2 || strategy == 4; }
// the stored parameter is the pair (theta, dtheta): B, C and the register variant
__host__ __device__ constexpr bool parameter_is_pair(int strategy) { return strategy == 1 || strategy == 2 || strategy == 4; }


// Algorithm 2 lines 10-12 for two parameters: the update delta from m, v (first component) and theta.
//
// FAST is chosen on the host when the bias corrections lie in [2^-100, 1] and 2^-54 <= eps <= 2^60
// (every practical setting).  Then (i) the two scalar divisions need no range test, (ii) the
// denominator is NaN, Inf or >= eps, hence a valid operand of div2_normal_divisor, and (iii) with
// epsilon outside the root a subnormal v-hat may be flushed by the root approximation: its root is
// below 2^-63 < ulp(eps)/2 and is absorbed by the addition of eps either way.
// With FAST the rare lanes are not answered here: they set bits in `suspect` (see the deferred
// forms above) and the caller repeats the vector with FAST = false, which never touches `suspect`.
template <bool FAST>
__device__ __forceinline__ bf2 update_ratio(bf2 m, bf2 v, const StepScalars& k, uint32_t& suspect) {
    bf2 mhat, vhat, den;
    if (FAST) {
        mhat = div2_by_scalar(m, k.rbc1);
        vhat = div2_by_scalar(v, k.rbc2);
        if (k.flags & 1u) den = sqrt2_flushing_deferred(add2(vhat, k.eps), suspect);   // v-hat + eps >= eps: never subnormal
        else den = add2(sqrt2_flushing_deferred(vhat, suspect), k.eps);
        return div2_normal_divisor_deferred(mhat, den, suspect);
    }
    mhat = div2_scalar(m, k.bc1, k.rbc1);
    vhat = div2_scalar(v, k.bc2, k.rbc2);
    if (k.flags & 1u) den = sqrt2(add2(vhat, k.eps));
    else den = add2(sqrt2(vhat), k.eps);
    return div2(mhat, den);
}

// What one step asked of two parameters: the update of line 12 and, when weight decay is applied
// by an addition of its own (Appendix D; flags bit 2), that decay term.
struct PairUpdate {
    bf2 delta, decay;
};

// Algorithm 2 lines 8-13 for two parameters; `s` is updated in place.
// STRATEGY: 0 = A, 1 = B, 2 = C, 3 = BF16-Kahan (Appendix B; s.dth holds the compensation c).
// VARIANT kernels honour flags bit 1 (the parameter Grow uses TwoSum) and bit 2 (decay by its own
// addition); the others are compiled without either, so the common path carries no test for them.
template <int STRATEGY, bool FAST, bool VARIANT>
__device__ __forceinline__ PairUpdate adamw_pair(ElemState& s, bf2 g, const StepScalars& k, uint32_t& suspect) {
    // line 8
    s.m = add2(mul2(k.b1, s.m), mul2(k.c1, g));
    // line 9
    const bf2 tv = mul2(k.c2, mul2(g, g));
    if (STRATEGY == 2) {
        const bf2pair decayed = mcf_mul2(k.b2h, k.b2l, s.v, s.dv);
        const bf2pair nv = grow2(decayed.hi, decayed.lo, tv);
        s.v = nv.hi;
        s.dv = nv.lo;
    } else {
        s.v = add2(mul2(k.b2, s.v), tv);
    }
    // lines 10-12
    const bf2 r = update_ratio<FAST>(s.m, s.v, k, suspect);
    const bf2 w = mul2(k.lam, s.th);
    const bool split_decay = VARIANT && (k.flags & 4u) != 0;
    PairUpdate up;
    up.decay = split_decay ? mul2(k.neg_a, w) : 0u;
    up.delta = split_decay ? mul2(k.neg_a, r) : mul2(k.neg_a, add2(r, w));
    // line 13
    if (STRATEGY == 3) {
        const bf2 comp = add2(up.delta, s.dth);
        const bf2 th_new = add2(s.th, comp);
        s.dth = sub2(comp, sub2(th_new, s.th));
        s.th = th_new;
    } else if (STRATEGY == 0) {
        if (split_decay) s.th = add2(s.th, up.decay);
        s.th = add2(s.th, up.delta);
    } else {
        const bool two_sum = VARIANT && (k.flags & 2u) != 0;
        if (split_decay) {
            const bf2pair nd = two_sum ? grow_two_sum2(s.th, s.dth, up.decay) : grow2(s.th, s.dth, up.decay);
            s.th = nd.hi;
            s.dth = nd.lo;
        }
        const bf2pair nt = two_sum ? grow_two_sum2(s.th, s.dth, up.delta) : grow2(s.th, s.dth, up.delta);
        s.th = nt.hi;
        s.dth = nt.lo;
    }
    return up;
}

// EDQ contributions of two parameters (Eq. 2-3): differences, products and running sums in
// float, two lanes at a time (lane = half of the bf2).
struct EdqAcc {
    f32x2 dot, sq;
    uint32_t lost;
};

// `d` is the intended update as two floats; the stored parameter is (th, dth) when HAS_LO, else th alone.
// A parameter counts as lost (Definition 3.2; "not updated", Figure 3 left) when an update was intended
// and the effective update e of Eq. 2 is zero: the value theta + dtheta did not move, whether or not
// Grow re-split it over other components.  e is formed in float, differences first; for normalised
// pairs it is zero exactly when the real number is (each difference of two bfloat16 values is exact in
// float unless it is far too large for the other difference to cancel, and a float sum of two
// non-zero numbers is zero only when they are opposite).
template <bool HAS_LO>
__device__ __forceinline__ void edq_pair_f(EdqAcc& acc, bf2 th_old, bf2 dth_old, bf2 th_new, bf2 dth_new, f32x2 d) {
    f32x2 e = sub_f32x2(widen2(th_new), widen2(th_old));
    if (HAS_LO) e = add_f32x2(e, sub_f32x2(widen2(dth_new), widen2(dth_old)));
    acc.dot = fma_f32x2(d, e, acc.dot);
    acc.sq = fma_f32x2(d, d, acc.sq);
    acc.lost += (lo_of(d) != 0.0f && lo_of(e) == 0.0f) ? 1u : 0u;
    acc.lost += (hi_of(d) != 0.0f && hi_of(e) == 0.0f) ? 1u : 0u;
}
// The same with the two decisions taken on packed bfloat16 values.  `asked` is the intended update as
// a bfloat16 pair, zero where `d` is.  e is rounded to bfloat16 only to be compared with zero: every
// term is a multiple of 2^-133, so a non-zero e is at least the smallest bfloat16 subnormal and stays
// non-zero, a NaN stays NaN (equal to nothing), and zeros of either sign compare equal.
// acc.lost collects the two halves as packed 16-bit counts: see edq_lost_packed.
template <bool HAS_LO>
__device__ __forceinline__ void edq_pair_packed(EdqAcc& acc, bf2 th_old, bf2 dth_old, bf2 th_new, bf2 dth_new, f32x2 d,
                                                bf2 asked) {
    f32x2 e = sub_f32x2(widen2(th_new), widen2(th_old));
    if (HAS_LO) e = add_f32x2(e, sub_f32x2(widen2(dth_new), widen2(dth_old)));
    acc.dot = fma_f32x2(d, e, acc.dot);
    acc.sq = fma_f32x2(d, d, acc.sq);
    acc.lost += equal2(pack_rn2(e), 0u) & differs2(asked, 0u) & 0x00010001u;
}
// the count held in packed form by edq_pair_packed (at most 65535 pairs between two calls)
__device__ __forceinline__ uint32_t edq_lost_packed(const EdqAcc& a) { return (a.lost & 0xFFFFu) + (a.lost >> 16); }
template <bool HAS_LO>
__device__ __forceinline__ void edq_pair(EdqAcc& acc, bf2 th_old, bf2 dth_old, bf2 th_new, bf2 dth_new, bf2 delta) {
    edq_pair_f<HAS_LO>(acc, th_old, dth_old, th_new, dth_new, widen2(delta));
}
__device__ __forceinline__ float edq_dot(const EdqAcc& a) { return __fadd_rn(lo_of(a.dot), hi_of(a.dot)); }
__device__ __forceinline__ float edq_sq(const EdqAcc& a) { return __fadd_rn(lo_of(a.sq), hi_of(a.sq)); }

// ---- variant: float arithmetic in registers on option C's storage (strategy 4) -----------------
// One lane: widen, AdamW in IEEE single operations (the option-D comparator's order), split back
// into normalised bfloat16 pairs.  Returns the float update; the lane's five values are updated.
__device__ __forceinline__ uint32_t bf16_bits_rn(float x) {
    uint16_t h;
    asm("cvt.rn.bf16.f32 %0, %1;" : "=h"(h) : "f"(x));
    return h;
}
__device__ __forceinline__ float adamw_register_lane(uint32_t& th, uint32_t& dth, uint32_t& m, uint32_t& v, uint32_t& dv,
                                                     uint32_t g16, const FloatScalars& k, uint32_t flags) {
    auto w = [](uint32_t h) { return __uint_as_float(h << 16); };
    const float g = w(g16);
    const float x = __fadd_rn(w(th), w(dth));
    const float vv = __fadd_rn(w(v), w(dv));
    const float m_new = __fadd_rn(__fmul_rn(k.b1, w(m)), __fmul_rn(k.c1, g));
    const float v_new = __fadd_rn(__fmul_rn(k.b2, vv), __fmul_rn(k.c2, __fmul_rn(g, g)));
    const float mhat = __fdiv_rn(m_new, k.bc1);
    const float vhat = __fdiv_rn(v_new, k.bc2);
    const float den = (flags & 1u) ? __fsqrt_rn(__fadd_rn(vhat, k.eps)) : __fadd_rn(__fsqrt_rn(vhat), k.eps);
    const float u = __fadd_rn(__fdiv_rn(mhat, den), __fmul_rn(k.lam, x));
    const float delta = __fmul_rn(k.neg_a, u);
    const float x_new = __fadd_rn(x, delta);
    th = bf16_bits_rn(x_new);
    dth = bf16_bits_rn(__fsub_rn(x_new, w(th)));
    m = bf16_bits_rn(m_new);
    v = bf16_bits_rn(v_new);
    dv = bf16_bits_rn(__fsub_rn(v_new, w(v)));
    return delta;
}

}  // namespace collage
