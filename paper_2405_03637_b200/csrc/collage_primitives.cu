// Batched MCF primitives, single rounded operations and the stand-alone EDQ reduction.
// All kernels are elementwise grid-stride loops over 8-element vectors built on the same device
// functions as the fused step (mcf_device.cuh).
#include "host_common.cuh"
#include "mcf_device.cuh"

namespace collage {

void launch_edq_finalize(const EdqPartial* partials, int count, uint64_t n, collage_edq_t* out, cudaStream_t stream,
                         bool accumulate);

constexpr int kPrimThreads = 256;

enum PrimOp {
    PRIM_FAST_TWO_SUM, PRIM_TWO_SUM, PRIM_TWO_PROD, PRIM_GROW, PRIM_SCALING, PRIM_MUL, PRIM_RENORMALIZE,
    PRIM_ADD, PRIM_SUB, PRIM_MULR, PRIM_DIV, PRIM_SQRT, PRIM_FMA
};

struct PrimArgs {
    const uint16_t* in[4];
    uint16_t* out[2];
    uint64_t n;
    int aligned;
};

template <int OP>
struct PrimTraits;
#define COLLAGE_PRIM(op, nin, nout) \
    template <> struct PrimTraits<op> { static constexpr int kIn = nin, kOut = nout; };
COLLAGE_PRIM(PRIM_FAST_TWO_SUM, 2, 2)
COLLAGE_PRIM(PRIM_TWO_SUM, 2, 2)
COLLAGE_PRIM(PRIM_TWO_PROD, 2, 2)
COLLAGE_PRIM(PRIM_GROW, 3, 2)
COLLAGE_PRIM(PRIM_SCALING, 3, 2)
COLLAGE_PRIM(PRIM_MUL, 4, 2)
COLLAGE_PRIM(PRIM_RENORMALIZE, 2, 2)
COLLAGE_PRIM(PRIM_ADD, 2, 1)
COLLAGE_PRIM(PRIM_SUB, 2, 1)
COLLAGE_PRIM(PRIM_MULR, 2, 1)
COLLAGE_PRIM(PRIM_DIV, 2, 1)
COLLAGE_PRIM(PRIM_SQRT, 1, 1)
COLLAGE_PRIM(PRIM_FMA, 3, 1)
#undef COLLAGE_PRIM

template <int OP>
__device__ __forceinline__ bf2pair apply(bf2 a, bf2 b, bf2 c, bf2 d) {
    bf2pair r = {0u, 0u};
    switch (OP) {
        case PRIM_FAST_TWO_SUM: return fast_two_sum2(a, b);
        case PRIM_TWO_SUM: return two_sum2(a, b);
        case PRIM_TWO_PROD: return two_prod2(a, b);
        case PRIM_GROW: return grow2(a, b, c);
        case PRIM_SCALING: return scaling2(a, b, c);
        case PRIM_MUL: return mcf_mul2(a, b, c, d);
        case PRIM_RENORMALIZE: return fast_two_sum2(a, b);
        case PRIM_ADD: r.hi = add2(a, b); return r;
        case PRIM_SUB: r.hi = sub2(a, b); return r;
        case PRIM_MULR: r.hi = mul2(a, b); return r;
        case PRIM_DIV: r.hi = div2(a, b); return r;
        case PRIM_SQRT: r.hi = sqrt2(a); return r;
        case PRIM_FMA: r.hi = fma2(a, b, c); return r;
    }
    return r;
}

template <int OP>
__global__ void __launch_bounds__(kPrimThreads) primitive_kernel(const __grid_constant__ PrimArgs p) {
    constexpr int NIN = PrimTraits<OP>::kIn, NOUT = PrimTraits<OP>::kOut;
    const uint64_t nvec = (p.n + 7) >> 3;
    for (uint64_t i = blockIdx.x * static_cast<uint64_t>(kPrimThreads) + threadIdx.x; i < nvec;
         i += static_cast<uint64_t>(gridDim.x) * kPrimThreads) {
        const uint64_t off = i * 8;
        const uint64_t left = p.n - off;
        const int count = left < 8 ? static_cast<int>(left) : 8;
        const bool vec = p.aligned && count == 8;
        uint32_t in[4][4] = {};
#pragma unroll
        for (int a = 0; a < NIN; ++a) {
            if (vec) {
                const uint4 w = *reinterpret_cast<const uint4*>(p.in[a] + off);
                in[a][0] = w.x; in[a][1] = w.y; in[a][2] = w.z; in[a][3] = w.w;
            } else {
#pragma unroll
                for (int e = 0; e < 8; ++e)
                    if (e < count) in[a][e >> 1] |= static_cast<uint32_t>(p.in[a][off + e]) << (16 * (e & 1));
            }
        }
        uint32_t out[2][4];
#pragma unroll
        for (int j = 0; j < 4; ++j) {
            const bf2pair r = apply<OP>(in[0][j], in[1][j], in[2][j], in[3][j]);
            out[0][j] = r.hi;
            out[1][j] = r.lo;
        }
#pragma unroll
        for (int o = 0; o < NOUT; ++o) {
            if (vec) {
                *reinterpret_cast<uint4*>(p.out[o] + off) = make_uint4(out[o][0], out[o][1], out[o][2], out[o][3]);
            } else {
#pragma unroll
                for (int e = 0; e < 8; ++e)
                    if (e < count) p.out[o][off + e] = static_cast<uint16_t>(out[o][e >> 1] >> (16 * (e & 1)));
            }
        }
    }
}

// A thread reads all of its inputs before it writes, and no other thread touches its 8
// elements, so an output may be exactly one of the inputs.  Any other overlap is rejected.
static collage_status_t check_prim(const PrimArgs& p, int nin, int nout) {
    for (int a = 0; a < nin; ++a)
        if (!p.in[a]) return COLLAGE_ERR_NULL;
    for (int o = 0; o < nout; ++o)
        if (!p.out[o]) return COLLAGE_ERR_NULL;
    const uint64_t bytes = 2 * p.n;
    auto overlaps = [bytes](const void* x, const void* y) {
        const uintptr_t a = reinterpret_cast<uintptr_t>(x), b = reinterpret_cast<uintptr_t>(y);
        return a != b && a < b + bytes && b < a + bytes;
    };
    for (int o = 0; o < nout; ++o) {
        for (int a = 0; a < nin; ++a)
            if (overlaps(p.out[o], p.in[a])) return COLLAGE_ERR_ALIAS;
        for (int o2 = o + 1; o2 < nout; ++o2)
            if (p.out[o] == p.out[o2] || overlaps(p.out[o], p.out[o2])) return COLLAGE_ERR_ALIAS;
    }
    return COLLAGE_OK;
}

template <int OP>
static collage_status_t run_prim(PrimArgs p, void* stream) {
    constexpr int NIN = PrimTraits<OP>::kIn, NOUT = PrimTraits<OP>::kOut;
    if (p.n > (1ull << 62)) return COLLAGE_ERR_ARG;
    collage_status_t st = check_prim(p, NIN, NOUT);
    if (st != COLLAGE_OK) return st;
    DeviceInfo dev;
    st = current_device(&dev);
    if (st != COLLAGE_OK) return st;
    if (p.n == 0) return COLLAGE_OK;
    uintptr_t bits = 0;
    for (int a = 0; a < NIN; ++a) bits |= reinterpret_cast<uintptr_t>(p.in[a]);
    for (int o = 0; o < NOUT; ++o) bits |= reinterpret_cast<uintptr_t>(p.out[o]);
    p.aligned = (bits & 15u) == 0;
    const uint64_t nvec = (p.n + 7) >> 3;
    uint64_t grid = (nvec + kPrimThreads - 1) / kPrimThreads;
    const uint64_t cap = static_cast<uint64_t>(dev.sm_count) * 16;
    if (grid > cap) grid = cap;
    primitive_kernel<OP><<<static_cast<unsigned>(grid), kPrimThreads, 0, static_cast<cudaStream_t>(stream)>>>(p);
    return cudaGetLastError() == cudaSuccess ? COLLAGE_OK : COLLAGE_ERR_CUDA;
}

static PrimArgs make_args(const void* a, const void* b, const void* c, const void* d, void* o0, void* o1, uint64_t n) {
    PrimArgs p{};
    p.in[0] = static_cast<const uint16_t*>(a);
    p.in[1] = static_cast<const uint16_t*>(b);
    p.in[2] = static_cast<const uint16_t*>(c);
    p.in[3] = static_cast<const uint16_t*>(d);
    p.out[0] = static_cast<uint16_t*>(o0);
    p.out[1] = static_cast<uint16_t*>(o1);
    p.n = n;
    return p;
}

// ------------------------------------------------------------------- EDQ ---

struct EdqArgs {
    const uint16_t* old_hi;
    const uint16_t* old_lo;
    const uint16_t* new_hi;
    const uint16_t* new_lo;
    const uint16_t* delta;
    uint64_t n;
    int aligned;
    EdqPartial* partials;
};

template <bool HAS_LO>
__global__ void __launch_bounds__(kPrimThreads) edq_kernel(const __grid_constant__ EdqArgs p) {
    double dot = 0.0, sq = 0.0;
    unsigned long long lost = 0;
    const uint64_t nvec = (p.n + 7) >> 3;
    for (uint64_t i = blockIdx.x * static_cast<uint64_t>(kPrimThreads) + threadIdx.x; i < nvec;
         i += static_cast<uint64_t>(gridDim.x) * kPrimThreads) {
        const uint64_t off = i * 8;
        const uint64_t left = p.n - off;
        const int count = left < 8 ? static_cast<int>(left) : 8;
        const bool vec = p.aligned && count == 8;
        const uint16_t* src[5] = {p.old_hi, p.old_lo, p.new_hi, p.new_lo, p.delta};
        uint32_t w[5][4] = {};
#pragma unroll
        for (int a = 0; a < 5; ++a) {
            if (!HAS_LO && (a == 1 || a == 3)) continue;
            if (vec) {
                const uint4 q = *reinterpret_cast<const uint4*>(src[a] + off);
                w[a][0] = q.x; w[a][1] = q.y; w[a][2] = q.z; w[a][3] = q.w;
            } else {
#pragma unroll
                for (int e = 0; e < 8; ++e)
                    if (e < count) w[a][e >> 1] |= static_cast<uint32_t>(src[a][off + e]) << (16 * (e & 1));
            }
        }
        EdqAcc acc = {0ull, 0ull, 0u};
#pragma unroll
        for (int j = 0; j < 4; ++j) edq_pair<HAS_LO>(acc, w[0][j], w[1][j], w[2][j], w[3][j], w[4][j]);
        dot += static_cast<double>(edq_dot(acc));
        sq += static_cast<double>(edq_sq(acc));
        lost += acc.lost;
    }
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) {
        dot += __shfl_down_sync(0xFFFFFFFFu, dot, o);
        sq += __shfl_down_sync(0xFFFFFFFFu, sq, o);
        lost += __shfl_down_sync(0xFFFFFFFFu, lost, o);
    }
    __shared__ double s_dot[kPrimThreads / 32], s_sq[kPrimThreads / 32];
    __shared__ unsigned long long s_lost[kPrimThreads / 32];
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    if (lane == 0) {
        s_dot[warp] = dot;
        s_sq[warp] = sq;
        s_lost[warp] = lost;
    }
    __syncthreads();
    if (threadIdx.x == 0) {
        double d = 0.0, q = 0.0;
        unsigned long long l = 0;
#pragma unroll
        for (int x = 0; x < kPrimThreads / 32; ++x) {
            d += s_dot[x];
            q += s_sq[x];
            l += s_lost[x];
        }
        p.partials[blockIdx.x] = EdqPartial{d, q, l, 0ull};
    }
}

// ------------------------------------------------------------- self test ---
// Exhaustive comparison of the arithmetic realisations used by the kernels with references
// built from IEEE float/double arithmetic and one cvt.rn to bfloat16.

__device__ __forceinline__ bool same_or_both_nan(uint32_t x, uint32_t y) {
    const bool xn = (x & 0x7F80u) == 0x7F80u && (x & 0x7Fu), yn = (y & 0x7F80u) == 0x7F80u && (y & 0x7Fu);
    return x == y || (xn && yn);
}
__device__ __forceinline__ uint32_t mismatches(bf2 x, bf2 y) {
    return (same_or_both_nan(x & 0xFFFFu, y & 0xFFFFu) ? 0u : 1u) + (same_or_both_nan(x >> 16, y >> 16) ? 0u : 1u);
}
// exact product of two bfloat16 values rounded once: double product (exact), truncated to float
// with a sticky last bit (round to odd), then cvt.rn
__device__ __forceinline__ float product_round_to_odd(float a, float b) {
    const double p = static_cast<double>(a) * static_cast<double>(b);
    float f = __double2float_rz(p);
    if (static_cast<double>(f) != p && isfinite(f)) f = __uint_as_float(__float_as_uint(f) | 1u);
    return f;
}

__global__ void __launch_bounds__(256) selftest_kernel(unsigned long long* counts) {
    unsigned long long c_add = 0, c_sub = 0, c_mul = 0, c_div = 0, c_sdiv = 0;
    const uint64_t stride = static_cast<uint64_t>(gridDim.x) * blockDim.x;
    // every (a, b): a in the outer 16 bits, two consecutive b per item
    for (uint64_t i = blockIdx.x * static_cast<uint64_t>(blockDim.x) + threadIdx.x; i < (1ull << 31); i += stride) {
        const uint32_t a16 = static_cast<uint32_t>(i >> 15), b16 = static_cast<uint32_t>(i & 0x7FFFu) * 2u;
        const bf2 a = a16 | (a16 << 16), b = b16 | ((b16 + 1u) << 16);
        const float a0 = lo_f32(a), a1 = hi_f32(a), b0 = lo_f32(b), b1 = hi_f32(b);
        c_add += mismatches(add2(a, b), pack_rn(__fadd_rn(a1, b1), __fadd_rn(a0, b0)));
        c_sub += mismatches(sub2(a, b), pack_rn(__fsub_rn(a1, b1), __fsub_rn(a0, b0)));
        c_mul += mismatches(mul2(a, b), pack_rn(product_round_to_odd(a1, b1), product_round_to_odd(a0, b0)));
        c_div += mismatches(div2(a, b), div2_ieee(a, b));
        {
            // the branch-free quotient of the lean chain: a lane it does not flag must already be right,
            // for every divisor it admits (NaN, Inf, normal up to 2^126)
            uint32_t flag = 0u;
            const bf2 q = div2_normal_divisor_deferred(a, b, flag), ref = div2_ieee(a, b);
#pragma unroll
            for (int h = 0; h < 2; ++h) {
                const uint32_t d = (b >> (16 * h)) & 0x7FFFu, e = d >> 7;
                const bool admitted = e == 0xFFu || (e >= 1u && d <= 0x7E80u);
                const bool flagged = ((flag >> (16 * h)) & 0xFFFFu) != 0u;
                if (admitted && !flagged && !same_or_both_nan((q >> (16 * h)) & 0xFFFFu, (ref >> (16 * h)) & 0xFFFFu)) ++c_div;
            }
        }
        // scalar-divisor route: divisors are the positive normal values up to 1 (bias corrections live there)
        if (b16 >= 0x0080u && b16 + 1u <= 0x3F80u) {
            const double d0 = static_cast<double>(b0), d1 = static_cast<double>(b1);
            // the host vouches for divisors in [2^-100, 1]: the reciprocal is then used without any test
            const float r0 = (d0 >= 0x1p-100) ? static_cast<float>(1.0 / d0) : nanf("");
            const float r1 = (d1 >= 0x1p-100) ? static_cast<float>(1.0 / d1) : nanf("");
            const bf2 q0 = div2_scalar(a, b0, r0), q1 = div2_scalar(a, b1, r1);
            c_sdiv += mismatches((q0 & 0xFFFFu) | (q1 << 16), div2_ieee(a, b));
        }
    }
    unsigned long long c_sqrt = 0;
    for (uint64_t i = blockIdx.x * static_cast<uint64_t>(blockDim.x) + threadIdx.x; i < (1ull << 15); i += stride) {
        const uint32_t x = static_cast<uint32_t>(i) * 2u;
        const bf2 a = x | ((x + 1u) << 16);
        c_sqrt += mismatches(sqrt2(a), sqrt2_ieee(a));
        // the branch-free root of the lean chain: unflagged lanes are right, except that a positive
        // subnormal may come out as +0 (its contract)
        uint32_t flag = 0u;
        const bf2 s = sqrt2_flushing_deferred(a, flag), ref = sqrt2_ieee(a);
#pragma unroll
        for (int h = 0; h < 2; ++h) {
            const uint32_t in = (a >> (16 * h)) & 0xFFFFu, got = (s >> (16 * h)) & 0xFFFFu;
            const bool flagged = ((flag >> (16 * h)) & 0xFFFFu) != 0u;
            const bool flushed = in >= 0x0001u && in <= 0x007Fu && got == 0u;
            if (!flagged && !flushed && !same_or_both_nan(got, (ref >> (16 * h)) & 0xFFFFu)) ++c_sqrt;
        }
    }
    unsigned long long v[6] = {c_add, c_sub, c_mul, c_div, c_sqrt, c_sdiv};
#pragma unroll
    for (int k = 0; k < 6; ++k) {
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) v[k] += __shfl_down_sync(0xFFFFFFFFu, v[k], o);
        if ((threadIdx.x & 31) == 0 && v[k]) atomicAdd(&counts[k], v[k]);
    }
}

}  // namespace collage

using namespace collage;

extern "C" {

collage_status_t collage_fast_two_sum(const void* a, const void* b, void* hi, void* lo, uint64_t n, void* stream) {
    return run_prim<PRIM_FAST_TWO_SUM>(make_args(a, b, nullptr, nullptr, hi, lo, n), stream);
}
collage_status_t collage_two_sum(const void* a, const void* b, void* hi, void* lo, uint64_t n, void* stream) {
    return run_prim<PRIM_TWO_SUM>(make_args(a, b, nullptr, nullptr, hi, lo, n), stream);
}
collage_status_t collage_two_prod(const void* a, const void* b, void* hi, void* lo, uint64_t n, void* stream) {
    return run_prim<PRIM_TWO_PROD>(make_args(a, b, nullptr, nullptr, hi, lo, n), stream);
}
collage_status_t collage_grow(const void* x, const void* y, const void* a, void* u, void* v, uint64_t n, void* stream) {
    return run_prim<PRIM_GROW>(make_args(x, y, a, nullptr, u, v, n), stream);
}
collage_status_t collage_scaling(const void* v, const void* a1, const void* a2, void* x, void* e, uint64_t n,
                                 void* stream) {
    return run_prim<PRIM_SCALING>(make_args(v, a1, a2, nullptr, x, e, n), stream);
}
collage_status_t collage_mul(const void* a1, const void* a2, const void* b1, const void* b2, void* x, void* e,
                             uint64_t n, void* stream) {
    return run_prim<PRIM_MUL>(make_args(a1, a2, b1, b2, x, e, n), stream);
}
collage_status_t collage_renormalize(const void* hi_in, const void* lo_in, void* hi, void* lo, uint64_t n,
                                     void* stream) {
    return run_prim<PRIM_RENORMALIZE>(make_args(hi_in, lo_in, nullptr, nullptr, hi, lo, n), stream);
}

collage_status_t collage_rounded_op(int op, const void* a, const void* b, const void* c, void* out, uint64_t n,
                                    void* stream) {
    switch (op) {
        case 0: return run_prim<PRIM_ADD>(make_args(a, b, nullptr, nullptr, out, nullptr, n), stream);
        case 1: return run_prim<PRIM_SUB>(make_args(a, b, nullptr, nullptr, out, nullptr, n), stream);
        case 2: return run_prim<PRIM_MULR>(make_args(a, b, nullptr, nullptr, out, nullptr, n), stream);
        case 3: return run_prim<PRIM_DIV>(make_args(a, b, nullptr, nullptr, out, nullptr, n), stream);
        case 4: return run_prim<PRIM_SQRT>(make_args(a, nullptr, nullptr, nullptr, out, nullptr, n), stream);
        case 5: return run_prim<PRIM_FMA>(make_args(a, b, c, nullptr, out, nullptr, n), stream);
        default: return COLLAGE_ERR_ARG;
    }
}

collage_status_t collage_edq(const void* old_hi, const void* old_lo, const void* new_hi, const void* new_lo,
                             const void* delta, uint64_t n, collage_edq_t* out_dev, void* workspace,
                             size_t workspace_bytes, void* stream) {
    if (!old_hi || !new_hi || !delta || !out_dev) return COLLAGE_ERR_NULL;
    if ((old_lo == nullptr) != (new_lo == nullptr)) return COLLAGE_ERR_NULL;
    if (n > (1ull << 62)) return COLLAGE_ERR_ARG;
    if (!workspace || workspace_bytes < kWorkspaceBytes || (reinterpret_cast<uintptr_t>(workspace) & 15u))
        return COLLAGE_ERR_WORKSPACE;
    DeviceInfo dev;
    collage_status_t st = current_device(&dev);
    if (st != COLLAGE_OK) return st;
    EdqArgs p{};
    p.old_hi = static_cast<const uint16_t*>(old_hi);
    p.old_lo = static_cast<const uint16_t*>(old_lo);
    p.new_hi = static_cast<const uint16_t*>(new_hi);
    p.new_lo = static_cast<const uint16_t*>(new_lo);
    p.delta = static_cast<const uint16_t*>(delta);
    p.n = n;
    const uintptr_t bits = reinterpret_cast<uintptr_t>(old_hi) | reinterpret_cast<uintptr_t>(old_lo) |
                           reinterpret_cast<uintptr_t>(new_hi) | reinterpret_cast<uintptr_t>(new_lo) |
                           reinterpret_cast<uintptr_t>(delta);
    p.aligned = (bits & 15u) == 0;
    p.partials = static_cast<EdqPartial*>(workspace);
    cudaStream_t cs = static_cast<cudaStream_t>(stream);
    const uint64_t nvec = (n + 7) >> 3;
    uint64_t grid = (nvec + kPrimThreads - 1) / kPrimThreads;
    const uint64_t cap = static_cast<uint64_t>(dev.sm_count) * 8;
    if (grid > cap) grid = cap;
    if (grid > static_cast<uint64_t>(kMaxGrid)) grid = kMaxGrid;
    if (grid > 0) {
        if (old_lo) edq_kernel<true><<<static_cast<unsigned>(grid), kPrimThreads, 0, cs>>>(p);
        else edq_kernel<false><<<static_cast<unsigned>(grid), kPrimThreads, 0, cs>>>(p);
        if (cudaGetLastError() != cudaSuccess) return COLLAGE_ERR_CUDA;
    }
    launch_edq_finalize(p.partials, static_cast<int>(grid), n, out_dev, cs, false);
    return cudaGetLastError() == cudaSuccess ? COLLAGE_OK : COLLAGE_ERR_CUDA;
}

collage_status_t collage_selftest(uint64_t out_host[6], void* stream) {
    if (!out_host) return COLLAGE_ERR_NULL;
    DeviceInfo dev;
    const collage_status_t st = current_device(&dev);
    if (st != COLLAGE_OK) return st;
    cudaStream_t cs = static_cast<cudaStream_t>(stream);
    unsigned long long* counts = nullptr;
    if (cudaMalloc(&counts, 6 * sizeof(unsigned long long)) != cudaSuccess) return COLLAGE_ERR_CUDA;
    cudaError_t e = cudaMemsetAsync(counts, 0, 6 * sizeof(unsigned long long), cs);
    if (e == cudaSuccess) {
        selftest_kernel<<<dev.sm_count * 8, 256, 0, cs>>>(counts);
        e = cudaGetLastError();
    }
    if (e == cudaSuccess) e = cudaMemcpyAsync(out_host, counts, 6 * sizeof(unsigned long long), cudaMemcpyDeviceToHost, cs);
    if (e == cudaSuccess) e = cudaStreamSynchronize(cs);
    cudaFree(counts);
    return e == cudaSuccess ? COLLAGE_OK : COLLAGE_ERR_CUDA;
}

}  // extern "C"
