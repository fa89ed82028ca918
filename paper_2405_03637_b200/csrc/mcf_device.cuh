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
//   div, sqrt       : no bfloat16 instruction exists.  Operands are widened to float (exact),
//                     the IEEE-correct float result is formed (div.rn.f32 / sqrt.rn.f32), and
//                     rounded to bfloat16 with cvt.rn.bf16x2.f32.  The float result carries 24
//                     bits >= 2*8+2, so the second rounding cannot change the outcome for
//                     results in the normal range.
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

__device__ __forceinline__ bf2 div2(bf2 a, bf2 b) {
    return pack_rn(__fdiv_rn(hi_f32(a), hi_f32(b)), __fdiv_rn(lo_f32(a), lo_f32(b)));
}
__device__ __forceinline__ bf2 sqrt2(bf2 a) {
    return pack_rn(__fsqrt_rn(hi_f32(a)), __fsqrt_rn(lo_f32(a)));
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

// bfloat16 scalars of one step, each duplicated into both halves of a bf2 (Algorithm 2 line 1).
struct StepScalars {
    bf2 b1, c1;        // RN(beta1), RN(1-beta1)
    bf2 b2, c2;        // RN(beta2), RN(1-beta2)
    bf2 b2h, b2l;      // beta2 as a length-2 expansion (Table 1)
    bf2 bc1, bc2;      // RN(1-beta1^t), RN(1-beta2^t)
    bf2 neg_a;         // -RN(lr)
    bf2 lam;           // RN(weight_decay)
    bf2 eps;           // RN(eps)
    uint32_t flags;
};

struct ElemState {
    bf2 th, dth, m, v, dv;
};

// Algorithm 2 lines 8-13 for two parameters.  STRATEGY: 0 = A, 1 = B, 2 = C.  Returns the
// bfloat16 update of line 12; `s` is updated in place.
template <int STRATEGY>
__device__ __forceinline__ bf2 adamw_pair(ElemState& s, bf2 g, const StepScalars& k) {
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
    const bf2 mhat = div2(s.m, k.bc1);
    const bf2 vhat = div2(s.v, k.bc2);
    bf2 den;
    if (k.flags & 1u) den = sqrt2(add2(vhat, k.eps));
    else den = add2(sqrt2(vhat), k.eps);
    const bf2 r = div2(mhat, den);
    const bf2 u = add2(r, mul2(k.lam, s.th));
    const bf2 delta = mul2(k.neg_a, u);
    // line 13
    if (STRATEGY == 0) {
        s.th = add2(s.th, delta);
    } else {
        const bf2pair nt = grow2(s.th, s.dth, delta);
        s.th = nt.hi;
        s.dth = nt.lo;
    }
    return delta;
}

// EDQ contributions of two parameters (Eq. 2-3): products in float.
struct EdqAcc {
    float dot, sq;
    uint32_t lost;
};

template <bool HAS_LO>
__device__ __forceinline__ void edq_pair(EdqAcc& acc, bf2 th_old, bf2 dth_old, bf2 th_new, bf2 dth_new, bf2 delta) {
    const float d0 = lo_f32(delta), d1 = hi_f32(delta);
    const float o0 = lo_f32(th_old), o1 = hi_f32(th_old);
    const float n0 = lo_f32(th_new), n1 = hi_f32(th_new);
    float e0 = __fsub_rn(n0, o0), e1 = __fsub_rn(n1, o1);
    bool same0 = (n0 == o0), same1 = (n1 == o1);
    if (HAS_LO) {
        const float p0 = lo_f32(dth_old), p1 = hi_f32(dth_old);
        const float q0 = lo_f32(dth_new), q1 = hi_f32(dth_new);
        e0 = __fadd_rn(e0, __fsub_rn(q0, p0));
        e1 = __fadd_rn(e1, __fsub_rn(q1, p1));
        same0 = same0 && (q0 == p0);
        same1 = same1 && (q1 == p1);
    }
    acc.dot = __fadd_rn(acc.dot, __fadd_rn(__fmul_rn(d0, e0), __fmul_rn(d1, e1)));
    acc.sq = __fadd_rn(acc.sq, __fadd_rn(__fmul_rn(d0, d0), __fmul_rn(d1, d1)));
    acc.lost += (d0 != 0.0f && same0) ? 1u : 0u;
    acc.lost += (d1 != 0.0f && same1) ? 1u : 0u;
}

}  // namespace collage
