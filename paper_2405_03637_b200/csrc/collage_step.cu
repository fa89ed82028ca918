// Fused Collage AdamW step (Algorithm 2 lines 8-13 + EDQ, Eq. 2-3): one persistent kernel that
// streams every state array exactly once, plus the entry points that launch it.
//
// Work is cut into chunks of `chunk_elems` consecutive elements of one tensor.  Thread block b
// takes chunks b, b + grid, b + 2*grid, ...  The kernel (step_pipeline.cuh) moves tiles between
// global and shared memory with the bulk asynchronous copy engine; its threads compute out of
// shared memory, 8 consecutive elements (one 16-byte vector per state array) at a time.  Tensors
// whose pointers are not all 16-byte aligned, and the ragged end of a tensor, go through plain or
// element-wise accesses that feed the same arithmetic.  EDQ sums: float within a vector, double
// per thread, fixed-order tree per block, one partial per block, summed by the block that
// finishes last (edq_reduce.cuh): a step is one launch.
#include <mutex>

#include "host_common.cuh"
#include "edq_reduce.cuh"
#include "mcf_device.cuh"

// Geometry of the pipeline kernel.  Measured on B200 (2^30 parameters, Collage-plus with EDQ, median
// of 80 launches): 512 consumer threads + one producer warp, one block per SM, three stages of
// 4096-element tiles reached 6.47 TB/s; an earlier register-staged kernel (16-byte loads into
// registers, 6 blocks of 128 threads per SM) 6.07 TB/s; smaller tiles, more stages or two blocks
// per SM were slower; 8192-element tiles in two stages (the same bytes in flight) measured the same
// within the 1 % run-to-run noise.
// Six staged arrays (option C, the register variant):
#ifndef COLLAGE_PIPE_CONSUMERS
#define COLLAGE_PIPE_CONSUMERS 512
#endif
#ifndef COLLAGE_PIPE_VPT
#define COLLAGE_PIPE_VPT 1
#endif
#ifndef COLLAGE_PIPE_STAGES
#define COLLAGE_PIPE_STAGES 3
#endif
// five staged arrays (option B, BF16-Kahan):
#ifndef COLLAGE_PIPE_CONSUMERS_B
#define COLLAGE_PIPE_CONSUMERS_B COLLAGE_PIPE_CONSUMERS
#endif
#ifndef COLLAGE_PIPE_VPT_B
#define COLLAGE_PIPE_VPT_B COLLAGE_PIPE_VPT
#endif
#ifndef COLLAGE_PIPE_STAGES_B
#define COLLAGE_PIPE_STAGES_B COLLAGE_PIPE_STAGES
#endif
// Option A moves the fewest bytes per parameter, so its arithmetic weighs more: 768 consumers
// (6144-element tiles) measured 6.67 TB/s against 5.96 TB/s with 512.
#ifndef COLLAGE_PIPE_CONSUMERS_A
#define COLLAGE_PIPE_CONSUMERS_A 768
#endif
#ifndef COLLAGE_PIPE_VPT_A
#define COLLAGE_PIPE_VPT_A COLLAGE_PIPE_VPT
#endif
#ifndef COLLAGE_PIPE_STAGES_A
#define COLLAGE_PIPE_STAGES_A COLLAGE_PIPE_STAGES
#endif
#ifndef COLLAGE_PIPE_MINBLOCKS
#define COLLAGE_PIPE_MINBLOCKS 1
#endif

namespace collage {

constexpr uint32_t kDefaultChunk = 24576;   // a whole number of tiles for every precision option (6 x 4096, 4 x 6144)
// consumer threads, vectors per thread and tile, and stages of the pipeline kernel for a precision option
struct PipeGeometry {
    int consumers, vpt, stages;
};
constexpr PipeGeometry pipe_geometry(int strategy) {
    return strategy == 0 ? PipeGeometry{COLLAGE_PIPE_CONSUMERS_A, COLLAGE_PIPE_VPT_A, COLLAGE_PIPE_STAGES_A}
           : (strategy == 1 || strategy == 3)
               ? PipeGeometry{COLLAGE_PIPE_CONSUMERS_B, COLLAGE_PIPE_VPT_B, COLLAGE_PIPE_STAGES_B}
               : PipeGeometry{COLLAGE_PIPE_CONSUMERS, COLLAGE_PIPE_VPT, COLLAGE_PIPE_STAGES};
}
// Option C on LARGE parameter sets: two stages of 8192-element tiles (two vectors per consumer thread), the
// same shared memory within 33 %.  Fewer, larger copies in flight stream 1-2 % faster from 2^28 parameters on
// (measured, interleaved, on one device: 4.221 against 4.305 ms on 1.27 G parameters, 0.900 against 0.913 ms
// on 2^28), are equal at 2^25..2^27 and slower below (a tensor of a few million parameters has too few tiles
// per block for tiles twice as long).
#ifndef COLLAGE_LARGE_TILE_MIN_N
#define COLLAGE_LARGE_TILE_MIN_N (1ull << 27)
#endif
#ifndef COLLAGE_LARGE_CONSUMERS
#define COLLAGE_LARGE_CONSUMERS 512
#endif
#ifndef COLLAGE_LARGE_VPT
#define COLLAGE_LARGE_VPT 2
#endif
#ifndef COLLAGE_LARGE_STAGES
#define COLLAGE_LARGE_STAGES 2
#endif
constexpr PipeGeometry kLargeGeometry = {COLLAGE_LARGE_CONSUMERS, COLLAGE_LARGE_VPT, COLLAGE_LARGE_STAGES};
// elements per tile
constexpr uint32_t pipe_tile(int strategy, bool large = false) {
    return large ? static_cast<uint32_t>(kLargeGeometry.consumers) * 8u * static_cast<uint32_t>(kLargeGeometry.vpt)
                 : static_cast<uint32_t>(pipe_geometry(strategy).consumers) * 8u * static_cast<uint32_t>(pipe_geometry(strategy).vpt);
}

struct TensorRec {
    uint16_t* x_hi;
    uint16_t* x_lo;
    uint16_t* m;
    uint16_t* v_hi;
    uint16_t* v_lo;
    const uint16_t* grad;
    uint64_t n;
    uint32_t aligned;   // all present pointers are 16-byte aligned
    uint32_t pad;
};

struct ChunkRec {
    uint32_t tensor;
    uint32_t index;     // chunk number inside the tensor: elements [index*chunk_elems, ...)
};

struct StepParams {
    TensorRec flat;             // used when the kernel is instantiated FLAT
    const TensorRec* tensors;   // multi-tensor table (device)
    const ChunkRec* chunks;     // chunk table (device)
    uint64_t num_chunks;
    uint32_t chunk_elems;
    StepScalars k;
    EdqFinish fin;              // per-block partials, ticket and record of the EDQ reduction (EDQ kernels)
    EdqPartial* chunk_partials; // one per chunk (per-tensor EDQ), or nullptr
    const uint64_t* replica_bases;  // [num_replicas][num_plan_tensors] base addresses of theta replicas, or nullptr
    int num_replicas;
    int num_plan_tensors;
};

// ---- 16-byte streaming accesses for tiles that bypass the copy pipeline ---------------------
__device__ __forceinline__ uint4 ld_stream(const uint16_t* p) { return __ldcs(reinterpret_cast<const uint4*>(p)); }
__device__ __forceinline__ void st_stream(uint16_t* p, const uint4& v) { __stcs(reinterpret_cast<uint4*>(p), v); }

// element-wise gather/scatter of up to 8 bfloat16 values into / out of four packed registers
__device__ __forceinline__ uint4 ld_elems(const uint16_t* p, int count) {
    uint32_t w[4] = {0u, 0u, 0u, 0u};
#pragma unroll
    for (int e = 0; e < 8; ++e)
        if (e < count) w[e >> 1] |= static_cast<uint32_t>(p[e]) << (16 * (e & 1));
    return make_uint4(w[0], w[1], w[2], w[3]);
}
__device__ __forceinline__ void st_elems(uint16_t* p, const uint4& v, int count) {
    const uint32_t w[4] = {v.x, v.y, v.z, v.w};
#pragma unroll
    for (int e = 0; e < 8; ++e)
        if (e < count) p[e] = static_cast<uint16_t>(w[e >> 1] >> (16 * (e & 1)));
}

struct Vec {
    uint4 th, dth, m, v, dv, g;
};

// The arithmetic of 8 parameters held in registers, every operand answered in place (the rare
// lanes by branches).  `valid` < 8 masks padded lanes out of EDQ.  FAST as in update_ratio, except
// that a lane it cannot answer is NOT repeated here: callers that pass FAST = true use
// compute_vec_fast below instead.
template <int STRATEGY, bool EDQ, bool VARIANT = false>
__device__ __forceinline__ void compute_vec(Vec& s, const StepScalars& k, int valid, double& dot, double& sq,
                                            uint32_t& lost) {
#ifdef COLLAGE_DATA_MOVEMENT_ONLY
    return;     // measurement build: every array goes through the pipeline unchanged
#endif
    uint32_t* th = reinterpret_cast<uint32_t*>(&s.th);
    uint32_t* dth = reinterpret_cast<uint32_t*>(&s.dth);
    uint32_t* m = reinterpret_cast<uint32_t*>(&s.m);
    uint32_t* v = reinterpret_cast<uint32_t*>(&s.v);
    uint32_t* dv = reinterpret_cast<uint32_t*>(&s.dv);
    const uint32_t* g = reinterpret_cast<const uint32_t*>(&s.g);
    EdqAcc acc = {0ull, 0ull, 0u};
    if constexpr (STRATEGY == 4) {
        // float arithmetic in registers: lane by lane, then the same EDQ terms on the stored pairs
#pragma unroll
        for (int j = 0; j < 4; ++j) {
            const bf2 th_old = th[j], dth_old = dth[j];
            uint32_t lane[2][5];
            float delta[2];
#pragma unroll
            for (int h = 0; h < 2; ++h) {
                const int sh = 16 * h;
                lane[h][0] = (th[j] >> sh) & 0xFFFFu;
                lane[h][1] = (dth[j] >> sh) & 0xFFFFu;
                lane[h][2] = (m[j] >> sh) & 0xFFFFu;
                lane[h][3] = (v[j] >> sh) & 0xFFFFu;
                lane[h][4] = (dv[j] >> sh) & 0xFFFFu;
                delta[h] = adamw_register_lane(lane[h][0], lane[h][1], lane[h][2], lane[h][3], lane[h][4],
                                               (g[j] >> sh) & 0xFFFFu, k.f, k.flags);
            }
            th[j] = lane[0][0] | (lane[1][0] << 16);
            dth[j] = lane[0][1] | (lane[1][1] << 16);
            m[j] = lane[0][2] | (lane[1][2] << 16);
            v[j] = lane[0][3] | (lane[1][3] << 16);
            dv[j] = lane[0][4] | (lane[1][4] << 16);
            if (EDQ) {
                bf2 th_new = th[j], dth_new = dth[j];
                const int lanes = valid - 2 * j;            // padded lanes hold zeros on input
                if (lanes < 2) {
                    const uint32_t mask = lanes == 1 ? 0x0000FFFFu : 0u;
                    th_new &= mask;
                    dth_new &= mask;
                    if (lanes < 2) delta[1] = 0.0f;
                    if (lanes < 1) delta[0] = 0.0f;
                }
                f32x2 d;
                asm("mov.b64 %0, {%1, %2};" : "=l"(d) : "f"(delta[0]), "f"(delta[1]));
                edq_pair_f<true>(acc, th_old, dth_old, th_new, dth_new, d);
            }
        }
    } else {
        uint32_t unused = 0u;
#pragma unroll
        for (int j = 0; j < 4; ++j) {
            ElemState e;
            e.th = th[j];
            e.dth = stores_x_lo(STRATEGY) ? dth[j] : 0u;   // delta-theta (B, C) or the Kahan compensation
            e.m = m[j];
            e.v = v[j];
            e.dv = stores_v_lo(STRATEGY) ? dv[j] : 0u;
            const bf2 th_old = e.th, dth_old = e.dth;
            const PairUpdate up = adamw_pair<STRATEGY, false, VARIANT>(e, g[j], k, unused);
            th[j] = e.th;
            m[j] = e.m;
            v[j] = e.v;
            if (stores_x_lo(STRATEGY)) dth[j] = e.dth;
            if (stores_v_lo(STRATEGY)) dv[j] = e.dv;
            if (EDQ) {
                bf2 th_new = e.th, dth_new = e.dth, delta = up.delta, decay = up.decay;
                if (valid < 8) {            // padded lanes hold zeros on input; keep them out of the sums
                    const int lanes = valid - 2 * j;
                    const uint32_t mask = lanes >= 2 ? 0xFFFFFFFFu : (lanes == 1 ? 0x0000FFFFu : 0u);
                    delta &= mask;
                    decay &= mask;
                    th_new &= mask;
                    dth_new &= mask;
                }
                // intended update: line 12, plus the separate decay term when there is one
                f32x2 d = widen2(delta);
                if (VARIANT && (k.flags & 4u)) d = add_f32x2(d, widen2(decay));
                // the stored parameter is the pair for options B and C, theta alone for A and Kahan
                edq_pair_f<parameter_is_pair(STRATEGY)>(acc, th_old, dth_old, th_new, dth_new, d);
            }
        }
    }
    if (EDQ) {
        dot += static_cast<double>(edq_dot(acc));
        sq += static_cast<double>(edq_sq(acc));
        lost += acc.lost;
    }
}

// The same for a full vector on the host-validated fast chain, without a branch: returns nonzero
// when some lane holds a quotient or root that the fast chain cannot answer.  The caller then
// discards `s` and `acc` and repeats the vector with compute_vec.
template <int STRATEGY, bool EDQ, bool VARIANT = false>
__device__ __forceinline__ uint32_t compute_vec_fast(Vec& s, const StepScalars& k, double& dot, double& sq, uint32_t& lost) {
    static_assert(STRATEGY != 4, "the register variant has no fast chain");
#ifdef COLLAGE_DATA_MOVEMENT_ONLY
    return 0u;  // measurement build: every array goes through the pipeline unchanged
#endif
    uint32_t* th = reinterpret_cast<uint32_t*>(&s.th);
    uint32_t* dth = reinterpret_cast<uint32_t*>(&s.dth);
    uint32_t* m = reinterpret_cast<uint32_t*>(&s.m);
    uint32_t* v = reinterpret_cast<uint32_t*>(&s.v);
    uint32_t* dv = reinterpret_cast<uint32_t*>(&s.dv);
    const uint32_t* g = reinterpret_cast<const uint32_t*>(&s.g);
    EdqAcc acc = {0ull, 0ull, 0u};
    uint32_t suspect = 0u;
#pragma unroll
    for (int j = 0; j < 4; ++j) {
        ElemState e;
        e.th = th[j];
        e.dth = stores_x_lo(STRATEGY) ? dth[j] : 0u;
        e.m = m[j];
        e.v = v[j];
        e.dv = stores_v_lo(STRATEGY) ? dv[j] : 0u;
        const bf2 th_old = e.th, dth_old = e.dth;
        const PairUpdate up = adamw_pair<STRATEGY, true, VARIANT>(e, g[j], k, suspect);
        th[j] = e.th;
        m[j] = e.m;
        v[j] = e.v;
        if (stores_x_lo(STRATEGY)) dth[j] = e.dth;
        if (stores_v_lo(STRATEGY)) dv[j] = e.dv;
        if (EDQ) {
            f32x2 d = widen2(up.delta);
            bf2 asked = up.delta;
            if (VARIANT && (k.flags & 4u)) {
                d = add_f32x2(d, widen2(up.decay));
                asked = add2(up.delta, up.decay);       // zero exactly where the float sum is
            }
            edq_pair_packed<parameter_is_pair(STRATEGY)>(acc, th_old, dth_old, e.th, e.dth, d, asked);
        }
    }
    if (EDQ && suspect == 0u) {
        dot += static_cast<double>(edq_dot(acc));
        sq += static_cast<double>(edq_sq(acc));
        lost += edq_lost_packed(acc);
    }
    return suspect;
}

// One vector of a tile staged in shared memory: array a of the tile starts at tile + a * TILE, in
// the order theta, m, v, [delta-theta], [delta-v], g.
template <int STRATEGY, int TILE>
__device__ __forceinline__ Vec tile_vector_load(const uint16_t* tile) {
    Vec r;
    int a = 0;
    r.th = *reinterpret_cast<const uint4*>(tile + TILE * a++);
    r.m = *reinterpret_cast<const uint4*>(tile + TILE * a++);
    r.v = *reinterpret_cast<const uint4*>(tile + TILE * a++);
    if (stores_x_lo(STRATEGY)) r.dth = *reinterpret_cast<const uint4*>(tile + TILE * a++);
    if (stores_v_lo(STRATEGY)) r.dv = *reinterpret_cast<const uint4*>(tile + TILE * a++);
    r.g = *reinterpret_cast<const uint4*>(tile + TILE * a);
    return r;
}
template <int STRATEGY, int TILE>
__device__ __forceinline__ void tile_vector_store(uint16_t* tile, const Vec& r) {
    int a = 0;
    *reinterpret_cast<uint4*>(tile + TILE * a++) = r.th;
    *reinterpret_cast<uint4*>(tile + TILE * a++) = r.m;
    *reinterpret_cast<uint4*>(tile + TILE * a++) = r.v;
    if (stores_x_lo(STRATEGY)) *reinterpret_cast<uint4*>(tile + TILE * a++) = r.dth;
    if (stores_v_lo(STRATEGY)) *reinterpret_cast<uint4*>(tile + TILE * a++) = r.dv;
}

// A vector that compute_vec_fast gave up on, repeated in place in the tile by the careful routes.
// Out of line on purpose: it runs for a vanishing share of the vectors and must not weigh on the
// register allocation of the loop that calls it.
struct VecSums {
    double dot, sq;
    uint32_t lost;
};
template <int STRATEGY, bool EDQ, bool VARIANT, int TILE>
__device__ __noinline__ VecSums careful_vector_in_tile(uint16_t* tile, const StepScalars& k) {
    VecSums r = {0.0, 0.0, 0u};
    Vec v = tile_vector_load<STRATEGY, TILE>(tile);
    compute_vec<STRATEGY, EDQ, VARIANT>(v, k, 8, r.dot, r.sq, r.lost);
    tile_vector_store<STRATEGY, TILE>(tile, v);
    return r;
}

template <int STRATEGY>
__device__ __forceinline__ void load_vec(Vec& s, const TensorRec& t, uint64_t off) {
    s.th = ld_stream(t.x_hi + off);
    s.m = ld_stream(t.m + off);
    s.v = ld_stream(t.v_hi + off);
    s.g = ld_stream(t.grad + off);
    if (stores_x_lo(STRATEGY)) s.dth = ld_stream(t.x_lo + off);
    if (stores_v_lo(STRATEGY)) s.dv = ld_stream(t.v_lo + off);
}
template <int STRATEGY>
__device__ __forceinline__ void store_vec(const Vec& s, const TensorRec& t, uint64_t off) {
    st_stream(t.x_hi + off, s.th);
    st_stream(t.m + off, s.m);
    st_stream(t.v_hi + off, s.v);
    if (stores_x_lo(STRATEGY)) st_stream(t.x_lo + off, s.dth);
    if (stores_v_lo(STRATEGY)) st_stream(t.v_lo + off, s.dv);
}
template <int STRATEGY>
__device__ __forceinline__ void load_elems(Vec& s, const TensorRec& t, uint64_t off, int count) {
    s.th = ld_elems(t.x_hi + off, count);
    s.m = ld_elems(t.m + off, count);
    s.v = ld_elems(t.v_hi + off, count);
    s.g = ld_elems(t.grad + off, count);
    if (stores_x_lo(STRATEGY)) s.dth = ld_elems(t.x_lo + off, count);
    if (stores_v_lo(STRATEGY)) s.dv = ld_elems(t.v_lo + off, count);
}
template <int STRATEGY>
__device__ __forceinline__ void store_elems(const Vec& s, const TensorRec& t, uint64_t off, int count) {
    st_elems(t.x_hi + off, s.th, count);
    st_elems(t.m + off, s.m, count);
    st_elems(t.v_hi + off, s.v, count);
    if (stores_x_lo(STRATEGY)) st_elems(t.x_lo + off, s.dth, count);
    if (stores_v_lo(STRATEGY)) st_elems(t.v_lo + off, s.dv, count);
}

}  // namespace collage
#include "step_pipeline.cuh"
#include "step_direct.cuh"
namespace collage {

// Sums the per-block partials in a fixed order and writes the EDQ record (Eq. 3).
// With `accumulate` the sums are added to the record's current contents (a step issued in slabs).
__global__ void __launch_bounds__(256) edq_finalize_kernel(const EdqPartial* partials, int count, uint64_t n,
                                                           collage_edq_t* out, int accumulate) {
    __shared__ double s_dot[256], s_sq[256];
    __shared__ unsigned long long s_lost[256];
    double d = 0.0, q = 0.0;
    unsigned long long l = 0;
    for (int i = threadIdx.x; i < count; i += 256) {
        d += partials[i].dot;
        q += partials[i].sq;
        l += partials[i].lost;
    }
    s_dot[threadIdx.x] = d;
    s_sq[threadIdx.x] = q;
    s_lost[threadIdx.x] = l;
    __syncthreads();
    for (int o = 128; o > 0; o >>= 1) {
        if (threadIdx.x < o) {
            s_dot[threadIdx.x] += s_dot[threadIdx.x + o];
            s_sq[threadIdx.x] += s_sq[threadIdx.x + o];
            s_lost[threadIdx.x] += s_lost[threadIdx.x + o];
        }
        __syncthreads();
    }
    if (threadIdx.x == 0) {
        double dot = s_dot[0], sq = s_sq[0];
        unsigned long long lost = s_lost[0];
        unsigned long long fault = 0;
        if (accumulate) {
            dot += out->dot;
            sq += out->sumsq;
            lost += out->lost;
            n += out->n;
            fault = out->fault;
        }
        out->dot = dot;
        out->sumsq = sq;
        out->edq = sq > 0.0 ? dot / sqrt(sq) : 0.0;
        out->n = n;
        out->lost = lost;
        out->fault = fault;
    }
}

// Per-tensor EDQ: block t adds the per-chunk partials of tensor t (chunks first[t] .. first[t+1]-1)
// in a fixed order and writes record index[t]; a second, single-block kernel adds the records.
__global__ void __launch_bounds__(256) edq_per_tensor_kernel(const EdqPartial* chunk_partials, const uint64_t* first,
                                                             const uint32_t* index, const uint64_t* sizes,
                                                             collage_edq_t* out) {
    __shared__ double s_dot[256], s_sq[256];
    __shared__ unsigned long long s_lost[256];
    const uint64_t lo = first[blockIdx.x], hi = first[blockIdx.x + 1];
    double d = 0.0, q = 0.0;
    unsigned long long l = 0;
    for (uint64_t i = lo + threadIdx.x; i < hi; i += 256) {
        d += chunk_partials[i].dot;
        q += chunk_partials[i].sq;
        l += chunk_partials[i].lost;
    }
    s_dot[threadIdx.x] = d;
    s_sq[threadIdx.x] = q;
    s_lost[threadIdx.x] = l;
    __syncthreads();
    for (int o = 128; o > 0; o >>= 1) {
        if (threadIdx.x < o) {
            s_dot[threadIdx.x] += s_dot[threadIdx.x + o];
            s_sq[threadIdx.x] += s_sq[threadIdx.x + o];
            s_lost[threadIdx.x] += s_lost[threadIdx.x + o];
        }
        __syncthreads();
    }
    if (threadIdx.x == 0) {
        collage_edq_t r;
        r.dot = s_dot[0];
        r.sumsq = s_sq[0];
        r.edq = s_sq[0] > 0.0 ? s_dot[0] / sqrt(s_sq[0]) : 0.0;
        r.n = sizes[blockIdx.x];
        r.lost = s_lost[0];
        r.fault = *reinterpret_cast<const volatile unsigned int*>(&g_pipeline_fault);
        out[index[blockIdx.x]] = r;
    }
}

__global__ void __launch_bounds__(32) edq_sum_records_kernel(const collage_edq_t* records, int count, collage_edq_t* out) {
    if (threadIdx.x != 0) return;
    double d = 0.0, q = 0.0;
    unsigned long long l = 0, n = 0;
    for (int i = 0; i < count; ++i) {      // tensor order: deterministic
        d += records[i].dot;
        q += records[i].sumsq;
        l += records[i].lost;
        n += records[i].n;
    }
    out->dot = d;
    out->sumsq = q;
    out->edq = q > 0.0 ? d / sqrt(q) : 0.0;
    out->n = n;
    out->lost = l;
    out->fault = *reinterpret_cast<const volatile unsigned int*>(&g_pipeline_fault);
}

void launch_edq_finalize(const EdqPartial* partials, int count, uint64_t n, collage_edq_t* out, cudaStream_t stream,
                         bool accumulate) {
    edq_finalize_kernel<<<1, 256, 0, stream>>>(partials, count, n, out, accumulate ? 1 : 0);
}

// ---------------------------------------------------------------- host side ---

static bf2 dup(uint16_t h) { return static_cast<uint32_t>(h) | (static_cast<uint32_t>(h) << 16); }

static collage_status_t make_scalars(const collage_hyper_t* hyper, uint64_t step, StepScalars* k) {
    uint16_t s[11];
    const collage_status_t st = collage_derive_scalars(hyper, step, s);
    if (st != COLLAGE_OK) return st;
    k->b1 = dup(s[0]);
    k->c1 = dup(s[1]);
    k->b2 = dup(s[2]);
    k->c2 = dup(s[3]);
    k->b2h = dup(s[4]);
    k->b2l = dup(s[5]);
    // scalar divisors as floats, with a host-rounded reciprocal when it is safely normal
    auto reciprocal = [](double d) {
        return (d >= 0x1p-100 && d <= 0x1p100) ? static_cast<float>(1.0 / d) : std::nanf("");
    };
    k->bc1 = static_cast<float>(bf16_to_double(s[6]));
    k->bc2 = static_cast<float>(bf16_to_double(s[7]));
    k->rbc1 = reciprocal(bf16_to_double(s[6]));
    k->rbc2 = reciprocal(bf16_to_double(s[7]));
    k->neg_a = dup(s[8] ^ 0x8000u);
    k->lam = dup(s[9]);
    k->eps = dup(s[10]);
    k->flags = hyper->flags & 7u;          // the kernels know the arithmetic flags only
    {   // float scalars of the register variant: each expression in double, one cast
        const double t = static_cast<double>(step);
        k->f.b1 = static_cast<float>(hyper->beta1);
        k->f.c1 = static_cast<float>(1.0 - hyper->beta1);
        k->f.b2 = static_cast<float>(hyper->beta2);
        k->f.c2 = static_cast<float>(1.0 - hyper->beta2);
        k->f.bc1 = static_cast<float>(1.0 - std::pow(hyper->beta1, t));
        k->f.bc2 = static_cast<float>(1.0 - std::pow(hyper->beta2, t));
        k->f.neg_a = -static_cast<float>(hyper->lr);
        k->f.lam = static_cast<float>(hyper->weight_decay);
        k->f.eps = static_cast<float>(hyper->eps);
    }
    // the lean arithmetic chain of the kernel is valid for these ranges (every practical setting)
    const double bc1 = bf16_to_double(s[6]), bc2 = bf16_to_double(s[7]), eps = bf16_to_double(s[10]);
    k->fast = (bc1 >= 0x1p-100 && bc1 <= 1.0 && bc2 >= 0x1p-100 && bc2 <= 1.0 && eps >= 0x1p-54 && eps <= 0x1p60) ? 1u : 0u;
#ifdef COLLAGE_IEEE_DIV_SQRT
    k->fast = 0u;
#endif
    return COLLAGE_OK;
}

template <int STRATEGY, bool EDQ, bool FLAT, bool FAST, bool PER_CHUNK = false, bool VARIANT = false, bool LARGE = false>
static cudaError_t launch_step(const StepParams& p, int sm_count, cudaStream_t stream, int* grid_out) {
    constexpr PipeGeometry G = LARGE ? kLargeGeometry : pipe_geometry(STRATEGY);
    constexpr int CONSUMERS = G.consumers;
    constexpr int VPT = G.vpt, STAGES = G.stages;
    auto kernel = adamw_step_pipeline_kernel<STRATEGY, EDQ, FLAT, FAST, CONSUMERS, VPT, STAGES, PER_CHUNK, VARIANT>;
    constexpr size_t smem = sizeof(PipeSmem<CONSUMERS, VPT, STAGES, STRATEGY>) + 128;
    constexpr int threads = CONSUMERS + 32;
    // per instantiation and per device: the shared-memory opt-in is a per-device function attribute.
    // Host threads that race on the first call each set the same attribute and store the same number.
    static std::atomic<int> per_device[64];
    int device = 0;
    if (cudaGetDevice(&device) != cudaSuccess || device < 0 || device >= 64) return cudaErrorInvalidDevice;
    int blocks_per_sm = per_device[device].load(std::memory_order_acquire);
    if (blocks_per_sm == 0) {
        cudaError_t e = cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, static_cast<int>(smem));
        if (e != cudaSuccess) return e;
        int b = 0;
        e = cudaOccupancyMaxActiveBlocksPerMultiprocessor(&b, kernel, threads, smem);
        if (e != cudaSuccess) return e;
        blocks_per_sm = b > 0 ? b : 1;
        per_device[device].store(blocks_per_sm, std::memory_order_release);
    }
    uint64_t grid = static_cast<uint64_t>(sm_count) * blocks_per_sm;
    if (grid > p.num_chunks) grid = p.num_chunks;
    if (grid > static_cast<uint64_t>(kMaxGrid)) grid = kMaxGrid;
    *grid_out = static_cast<int>(grid);
    kernel<<<static_cast<unsigned>(grid), threads, smem, stream>>>(p);
    return cudaGetLastError();
}

template <bool FLAT, bool FAST>
static cudaError_t dispatch_step2(const StepParams& p, int strategy, bool edq, int sm_count, cudaStream_t stream,
                                  int* grid_out, bool large) {
    if (large && strategy == 2)
        return edq ? launch_step<2, true, FLAT, FAST, false, false, true>(p, sm_count, stream, grid_out)
                   : launch_step<2, false, FLAT, FAST, false, false, true>(p, sm_count, stream, grid_out);
    switch (strategy * 2 + (edq ? 1 : 0)) {
        case 0: return launch_step<0, false, FLAT, FAST>(p, sm_count, stream, grid_out);
        case 1: return launch_step<0, true, FLAT, FAST>(p, sm_count, stream, grid_out);
        case 2: return launch_step<1, false, FLAT, FAST>(p, sm_count, stream, grid_out);
        case 3: return launch_step<1, true, FLAT, FAST>(p, sm_count, stream, grid_out);
        case 4: return launch_step<2, false, FLAT, FAST>(p, sm_count, stream, grid_out);
        case 5: return launch_step<2, true, FLAT, FAST>(p, sm_count, stream, grid_out);
        case 6: return launch_step<3, false, FLAT, FAST>(p, sm_count, stream, grid_out);
        case 7: return launch_step<3, true, FLAT, FAST>(p, sm_count, stream, grid_out);
        case 8: return launch_step<4, false, FLAT, false>(p, sm_count, stream, grid_out);   // no bfloat16 chain: FAST is moot
        default: return launch_step<4, true, FLAT, false>(p, sm_count, stream, grid_out);
    }
}
// multi-tensor step with one EDQ record per chunk
static cudaError_t dispatch_step_per_chunk(const StepParams& p, int strategy, int sm_count, cudaStream_t stream,
                                           int* grid_out, bool large) {
    if (large && strategy == 2)
        return p.k.fast ? launch_step<2, true, false, true, true, false, true>(p, sm_count, stream, grid_out)
                        : launch_step<2, true, false, false, true, false, true>(p, sm_count, stream, grid_out);
    switch (strategy * 2 + (p.k.fast ? 1 : 0)) {
        case 0: return launch_step<0, true, false, false, true>(p, sm_count, stream, grid_out);
        case 1: return launch_step<0, true, false, true, true>(p, sm_count, stream, grid_out);
        case 2: return launch_step<1, true, false, false, true>(p, sm_count, stream, grid_out);
        case 3: return launch_step<1, true, false, true, true>(p, sm_count, stream, grid_out);
        case 4: return launch_step<2, true, false, false, true>(p, sm_count, stream, grid_out);
        case 5: return launch_step<2, true, false, true, true>(p, sm_count, stream, grid_out);
        case 6: return launch_step<3, true, false, false, true>(p, sm_count, stream, grid_out);
        case 7: return launch_step<3, true, false, true, true>(p, sm_count, stream, grid_out);
        default: return launch_step<4, true, false, false, true>(p, sm_count, stream, grid_out);
    }
}

// steps with a variant flag set (TwoSum Grow, decay by its own addition): options A, B, C
template <bool FLAT, bool FAST>
static cudaError_t dispatch_variant(const StepParams& p, int strategy, bool edq, int sm_count, cudaStream_t stream,
                                    int* grid_out) {
    switch (strategy * 2 + (edq ? 1 : 0)) {
        case 0: return launch_step<0, false, FLAT, FAST, false, true>(p, sm_count, stream, grid_out);
        case 1: return launch_step<0, true, FLAT, FAST, false, true>(p, sm_count, stream, grid_out);
        case 2: return launch_step<1, false, FLAT, FAST, false, true>(p, sm_count, stream, grid_out);
        case 3: return launch_step<1, true, FLAT, FAST, false, true>(p, sm_count, stream, grid_out);
        case 4: return launch_step<2, false, FLAT, FAST, false, true>(p, sm_count, stream, grid_out);
        case 5: return launch_step<2, true, FLAT, FAST, false, true>(p, sm_count, stream, grid_out);
        default: return cudaErrorInvalidValue;
    }
}

// Does a Collage-plus step over `n` parameters take the large tiles?  `choice` = the kernel-choice flags.
static bool takes_large_tiles(int strategy, uint32_t arithmetic_flags, uint32_t choice, uint64_t n) {
    if (strategy != COLLAGE_PLUS || (arithmetic_flags & (COLLAGE_FLAG_TWOSUM_GROW | COLLAGE_FLAG_DECAY_BY_GROW))) return false;
    if (choice & COLLAGE_FLAG_LARGE_TILES) return true;
    return !(choice & COLLAGE_FLAG_PIPELINE_KERNEL) && n >= COLLAGE_LARGE_TILE_MIN_N;
}

template <bool FLAT>
static cudaError_t dispatch_step(const StepParams& p, int strategy, bool edq, int sm_count, cudaStream_t stream,
                                 int* grid_out, bool large = false) {
    if (p.k.flags & (COLLAGE_FLAG_TWOSUM_GROW | COLLAGE_FLAG_DECAY_BY_GROW))
        return p.k.fast ? dispatch_variant<FLAT, true>(p, strategy, edq, sm_count, stream, grid_out)
                        : dispatch_variant<FLAT, false>(p, strategy, edq, sm_count, stream, grid_out);
    return p.k.fast ? dispatch_step2<FLAT, true>(p, strategy, edq, sm_count, stream, grid_out, large)
                    : dispatch_step2<FLAT, false>(p, strategy, edq, sm_count, stream, grid_out, large);
}

static bool aligned16(const void* p) { return (reinterpret_cast<uintptr_t>(p) & 15u) == 0; }

// ---- small flat tensors: the direct kernel (step_direct.cuh) ---------------------------------
// Flat tensors up to this many parameters take the direct kernel.  Measured on B200 (Collage-plus with
// EDQ, steps replayed from a CUDA graph, one device): 2^16 parameters 4.2 against 6.4 microseconds with the
// pipeline kernel, 2^20 9.3 against 10.7, 2^21 13.2 against 14.5, 2^22 20.9 against 21.1, 2^23 36.6 against 35.1.
#ifndef COLLAGE_DIRECT_MAX_N
#define COLLAGE_DIRECT_MAX_N (1ull << 21)
#endif

template <int STRATEGY, bool EDQ, bool FAST, bool VARIANT>
static cudaError_t launch_direct(const StepParams& p, int sm_count, cudaStream_t stream, int* grid_out) {
    auto kernel = adamw_step_direct_kernel<STRATEGY, EDQ, FAST, VARIANT>;
    static std::atomic<int> per_device[64];
    int device = 0;
    if (cudaGetDevice(&device) != cudaSuccess || device < 0 || device >= 64) return cudaErrorInvalidDevice;
    int blocks_per_sm = per_device[device].load(std::memory_order_acquire);
    if (blocks_per_sm == 0) {
        int b = 0;
        const cudaError_t e = cudaOccupancyMaxActiveBlocksPerMultiprocessor(&b, kernel, kDirectThreads, 0);
        if (e != cudaSuccess) return e;
        blocks_per_sm = b > 0 ? b : 1;
        per_device[device].store(blocks_per_sm, std::memory_order_release);
    }
    const uint64_t nvec = (p.flat.n + 7) >> 3;
    uint64_t grid = (nvec + kDirectThreads - 1) / kDirectThreads;
    const uint64_t resident = static_cast<uint64_t>(sm_count) * blocks_per_sm;
    if (grid > resident) grid = resident;
    if (grid > static_cast<uint64_t>(kMaxGrid)) grid = kMaxGrid;
    *grid_out = static_cast<int>(grid);
    kernel<<<static_cast<unsigned>(grid), kDirectThreads, 0, stream>>>(p);
    return cudaGetLastError();
}

template <bool FAST, bool VARIANT>
static cudaError_t dispatch_direct2(const StepParams& p, int strategy, bool edq, int sm_count, cudaStream_t stream,
                                    int* grid_out) {
    switch (strategy * 2 + (edq ? 1 : 0)) {
        case 0: return launch_direct<0, false, FAST, VARIANT>(p, sm_count, stream, grid_out);
        case 1: return launch_direct<0, true, FAST, VARIANT>(p, sm_count, stream, grid_out);
        case 2: return launch_direct<1, false, FAST, VARIANT>(p, sm_count, stream, grid_out);
        case 3: return launch_direct<1, true, FAST, VARIANT>(p, sm_count, stream, grid_out);
        case 4: return launch_direct<2, false, FAST, VARIANT>(p, sm_count, stream, grid_out);
        case 5: return launch_direct<2, true, FAST, VARIANT>(p, sm_count, stream, grid_out);
        default: break;
    }
    if constexpr (!VARIANT) {
        switch (strategy * 2 + (edq ? 1 : 0)) {
            case 6: return launch_direct<3, false, FAST, false>(p, sm_count, stream, grid_out);
            case 7: return launch_direct<3, true, FAST, false>(p, sm_count, stream, grid_out);
            case 8: return launch_direct<4, false, false, false>(p, sm_count, stream, grid_out);
            case 9: return launch_direct<4, true, false, false>(p, sm_count, stream, grid_out);
            default: break;
        }
    }
    return cudaErrorInvalidValue;
}

static cudaError_t dispatch_direct(const StepParams& p, int strategy, bool edq, int sm_count, cudaStream_t stream,
                                   int* grid_out) {
    const bool variant = (p.k.flags & (COLLAGE_FLAG_TWOSUM_GROW | COLLAGE_FLAG_DECAY_BY_GROW)) != 0;
    if (variant)
        return p.k.fast ? dispatch_direct2<true, true>(p, strategy, edq, sm_count, stream, grid_out)
                        : dispatch_direct2<false, true>(p, strategy, edq, sm_count, stream, grid_out);
    return p.k.fast ? dispatch_direct2<true, false>(p, strategy, edq, sm_count, stream, grid_out)
                    : dispatch_direct2<false, false>(p, strategy, edq, sm_count, stream, grid_out);
}

// Launches the flat (single tensor) step on device pointers; no-op for n == 0.
static cudaError_t launch_flat(void* x_hi, void* x_lo, void* m, void* v_hi, void* v_lo, const void* grad, uint64_t n,
                               const StepScalars& k, int strategy, const EdqFinish& fin, int sm_count,
                               cudaStream_t stream, int* grid_out, uint32_t kernel_choice = 0) {
    *grid_out = 0;
    if (n == 0) return cudaSuccess;
    StepParams p{};
    p.k = k;
    p.flat.x_hi = static_cast<uint16_t*>(x_hi);
    p.flat.x_lo = static_cast<uint16_t*>(x_lo);
    p.flat.m = static_cast<uint16_t*>(m);
    p.flat.v_hi = static_cast<uint16_t*>(v_hi);
    p.flat.v_lo = static_cast<uint16_t*>(v_lo);
    p.flat.grad = static_cast<const uint16_t*>(grad);
    p.flat.n = n;
    p.flat.aligned = aligned16(x_hi) && aligned16(x_lo) && aligned16(m) && aligned16(v_hi) && aligned16(v_lo) &&
                     aligned16(grad);
    // four tiles per chunk when there is plenty of work, one tile per chunk when the tensor is small,
    // so that every SM still gets a share
    const bool large = takes_large_tiles(strategy, k.flags, kernel_choice, n);
    const uint32_t tile = pipe_tile(strategy, large);
    uint32_t chunk = 4 * tile;
    if ((n + chunk - 1) / chunk < 4ull * static_cast<uint64_t>(sm_count)) chunk = tile;
    p.chunk_elems = chunk;
    p.num_chunks = (n + chunk - 1) / chunk;
    p.fin = fin;
    const bool direct = (kernel_choice & COLLAGE_FLAG_DIRECT_KERNEL) ||
                        (!(kernel_choice & (COLLAGE_FLAG_PIPELINE_KERNEL | COLLAGE_FLAG_LARGE_TILES)) && n <= COLLAGE_DIRECT_MAX_N);
    if (direct) return dispatch_direct(p, strategy, fin.out != nullptr, sm_count, stream, grid_out);
    return dispatch_step<true>(p, strategy, fin.out != nullptr, sm_count, stream, grid_out, large);
}

static collage_status_t check_common(const collage_hyper_t* hyper, uint64_t step, int strategy) {
    if (!hyper) return COLLAGE_ERR_NULL;
    if (step == 0) return COLLAGE_ERR_ARG;
    if (strategy < COLLAGE_BF16 || strategy > COLLAGE_PLUS_FP32_REGISTERS) return COLLAGE_ERR_ARG;
    if (!hyper_in_range(hyper)) return COLLAGE_ERR_ARG;
    if (hyper->flags & ~(COLLAGE_FLAG_EPS_INSIDE_SQRT | COLLAGE_FLAG_TWOSUM_GROW | COLLAGE_FLAG_DECAY_BY_GROW |
                         COLLAGE_FLAG_PIPELINE_KERNEL | COLLAGE_FLAG_DIRECT_KERNEL | COLLAGE_FLAG_LARGE_TILES))
        return COLLAGE_ERR_ARG;
    {   // at most one kernel choice
        const uint32_t choice = hyper->flags & (COLLAGE_FLAG_PIPELINE_KERNEL | COLLAGE_FLAG_DIRECT_KERNEL | COLLAGE_FLAG_LARGE_TILES);
        if (choice & (choice - 1)) return COLLAGE_ERR_ARG;
    }
    // TwoSum Grow needs a parameter pair (B, C); the Kahan comparator takes neither variant
    if ((hyper->flags & COLLAGE_FLAG_TWOSUM_GROW) && strategy != COLLAGE_LIGHT && strategy != COLLAGE_PLUS)
        return COLLAGE_ERR_ARG;
    if ((hyper->flags & COLLAGE_FLAG_DECAY_BY_GROW) && strategy >= COLLAGE_KAHAN) return COLLAGE_ERR_ARG;
    if (hyper->edq_out) {
        if (!hyper->workspace || hyper->workspace_bytes < kWorkspaceBytes) return COLLAGE_ERR_WORKSPACE;
        if (reinterpret_cast<uintptr_t>(hyper->workspace) & 15u) return COLLAGE_ERR_WORKSPACE;
        if (reinterpret_cast<uintptr_t>(hyper->edq_out) & 7u) return COLLAGE_ERR_ARG;     // a record of doubles
    }
    return COLLAGE_OK;
}

// where the pieces of the EDQ reduction live inside a workspace
static EdqFinish make_finish(void* workspace, void* record, uint64_t n, bool accumulate) {
    EdqFinish f{};
    if (record) {
        f.partials = static_cast<EdqPartial*>(workspace);
        f.ticket = reinterpret_cast<unsigned int*>(static_cast<char*>(workspace) + kTicketOffset);
        f.out = static_cast<collage_edq_t*>(record);
        f.n = n;
        f.accumulate = accumulate ? 1 : 0;
    }
    return f;
}

// byte ranges of the EDQ record and workspace of a call, for the overlap checks
static void push_edq_ranges(std::vector<ByteRange>& ranges, const collage_hyper_t* hyper) {
    if (hyper->edq_out) {
        push_bytes(ranges, hyper->edq_out, sizeof(collage_edq_t));
        push_bytes(ranges, hyper->workspace, kWorkspaceBytes);
    }
}

}  // namespace collage

namespace collage {
cudaError_t read_clear_fault32(unsigned int* out);
}
using namespace collage;

struct collage_plan {
    TensorRec* d_tensors = nullptr;
    ChunkRec* d_chunks = nullptr;
    uint64_t* d_first_chunk = nullptr;   // per non-empty tensor, plus an end marker
    uint64_t* d_sizes = nullptr;         // per non-empty tensor
    uint32_t* d_orig_index = nullptr;    // position of the tensor in the caller's array
    int num_given = 0;                   // length of the caller's array
    uint64_t* d_replica_bases = nullptr; // [num_replicas][num_tensors] (non-empty tensors only)
    int num_replicas = 0;
    std::vector<ByteRange> ranges;       // byte ranges of every array of the plan and of its replicas, sorted by address (overlap checks)
    std::vector<ByteRange> own_ranges;   // the same without the replicas
    std::vector<collage_tensor_t> given; // the caller's array, as given
    uint64_t num_chunks = 0;
    uint64_t num_elements = 0;
    uint32_t chunk_elems = 0;
    int num_tensors = 0;
    bool has_x_lo = true, has_v_lo = true;
    int device = 0;
};

// a plan's tables live on the device that was current when it was created
static bool plan_on_current_device(const collage_plan* plan) {
    int device = -1;
    return plan->num_tensors == 0 || (cudaGetDevice(&device) == cudaSuccess && device == plan->device);
}

extern "C" {

const char* collage_status_string(collage_status_t status) {
    switch (status) {
        case COLLAGE_OK: return "ok";
        case COLLAGE_ERR_NULL: return "a required pointer is NULL (or a component the strategy needs is missing)";
        case COLLAGE_ERR_ARG: return "invalid argument (step 0, unknown strategy or op, hyper-parameter out of range)";
        case COLLAGE_ERR_ALIAS: return "tensors overlap";
        case COLLAGE_ERR_ARCH: return "current device is not compute capability 10.x (sm_100a only, no fallback)";
        case COLLAGE_ERR_CUDA: return "CUDA runtime error";
        case COLLAGE_ERR_WORKSPACE: return "EDQ workspace missing, misaligned or too small";
        case COLLAGE_ERR_LIMIT: return "size beyond the fixed capacity of this entry point";
    }
    return "unknown status";
}

collage_status_t collage_derive_scalars(const collage_hyper_t* hyper, uint64_t step, uint16_t out[11]) {
    if (!hyper || !out) return COLLAGE_ERR_NULL;
    if (step == 0 || !hyper_in_range(hyper)) return COLLAGE_ERR_ARG;
    const double t = static_cast<double>(step);
    out[0] = double_to_bf16_rn(hyper->beta1);
    out[1] = double_to_bf16_rn(1.0 - hyper->beta1);
    out[2] = double_to_bf16_rn(hyper->beta2);
    out[3] = double_to_bf16_rn(1.0 - hyper->beta2);
    out[4] = out[2];
    out[5] = double_to_bf16_rn(hyper->beta2 - bf16_to_double(out[4]));
    out[6] = double_to_bf16_rn(1.0 - std::pow(hyper->beta1, t));
    out[7] = double_to_bf16_rn(1.0 - std::pow(hyper->beta2, t));
    out[8] = double_to_bf16_rn(hyper->lr);
    out[9] = double_to_bf16_rn(hyper->weight_decay);
    out[10] = double_to_bf16_rn(hyper->eps);
    return COLLAGE_OK;
}

size_t collage_workspace_bytes(uint64_t) { return kWorkspaceBytes; }

collage_status_t collage_workspace_init(void* workspace, size_t workspace_bytes, void* stream) {
    if (!workspace) return COLLAGE_ERR_NULL;
    if (workspace_bytes < kWorkspaceBytes || (reinterpret_cast<uintptr_t>(workspace) & 15u)) return COLLAGE_ERR_WORKSPACE;
    return cudaMemsetAsync(workspace, 0, kWorkspaceBytes, static_cast<cudaStream_t>(stream)) == cudaSuccess ? COLLAGE_OK
                                                                                                          : COLLAGE_ERR_CUDA;
}

collage_status_t collage_edq_combine(const collage_edq_t* parts, int count, collage_edq_t* out) {
    if (!out || (count > 0 && !parts)) return COLLAGE_ERR_NULL;
    if (count < 0) return COLLAGE_ERR_ARG;
    collage_edq_t r = {0.0, 0.0, 0.0, 0, 0, 0};
    for (int i = 0; i < count; ++i) {          // array order: the association of the sums is fixed
        r.dot += parts[i].dot;
        r.sumsq += parts[i].sumsq;
        r.n += parts[i].n;
        r.lost += parts[i].lost;
        if (!r.fault) r.fault = parts[i].fault;
    }
    r.edq = r.sumsq > 0.0 ? r.dot / std::sqrt(r.sumsq) : 0.0;     // Eq. 3
    *out = r;
    return COLLAGE_OK;
}

const char* collage_build_flavor(void) {
#ifdef COLLAGE_DATA_MOVEMENT_ONLY
    return "data-movement-only";
#else
    return "product";
#endif
}

collage_status_t collage_adamw_step(void* x_hi, void* x_lo, void* m, void* v_hi, void* v_lo, const void* grad,
                                    uint64_t n, const collage_hyper_t* hyper, uint64_t step,
                                    collage_strategy_t strategy, void* stream) {
    collage_status_t st = check_common(hyper, step, strategy);
    if (st != COLLAGE_OK) return st;
    if (!x_hi || !m || !v_hi || !grad) return COLLAGE_ERR_NULL;
    if ((strategy >= COLLAGE_LIGHT) != (x_lo != nullptr)) return x_lo ? COLLAGE_ERR_ARG : COLLAGE_ERR_NULL;
    if (stores_v_lo(strategy) != (v_lo != nullptr)) return v_lo ? COLLAGE_ERR_ARG : COLLAGE_ERR_NULL;
    if (n > (1ull << 62)) return COLLAGE_ERR_ARG;
    std::vector<ByteRange> ranges;
    for (const void* q : {static_cast<const void*>(x_hi), static_cast<const void*>(x_lo), static_cast<const void*>(m),
                          static_cast<const void*>(v_hi), static_cast<const void*>(v_lo), grad})
        push_range(ranges, q, n);
    push_edq_ranges(ranges, hyper);
    if (any_overlap(ranges)) return COLLAGE_ERR_ALIAS;
    DeviceInfo dev;
    st = current_device(&dev);
    if (st != COLLAGE_OK) return st;
    cudaStream_t cs = static_cast<cudaStream_t>(stream);

    StepScalars k;
    st = make_scalars(hyper, step, &k);
    if (st != COLLAGE_OK) return st;
    const bool edq = hyper->edq_out != nullptr;
    int grid = 0;
    if (launch_flat(x_hi, x_lo, m, v_hi, v_lo, grad, n, k, strategy, make_finish(hyper->workspace, hyper->edq_out, n, false),
                    dev.sm_count, cs, &grid, hyper->flags) != cudaSuccess)
        return COLLAGE_ERR_CUDA;
    if (edq && grid == 0) {        // nothing was launched (n == 0): the record still has to say so
        launch_edq_finalize(static_cast<EdqPartial*>(hyper->workspace), 0, 0, static_cast<collage_edq_t*>(hyper->edq_out), cs, false);
        if (cudaGetLastError() != cudaSuccess) return COLLAGE_ERR_CUDA;
    }
    return COLLAGE_OK;
}

collage_status_t collage_plan_create(const collage_tensor_t* tensors, int num, uint32_t chunk_elems,
                                     collage_plan_t** out_plan) {
    if (!out_plan) return COLLAGE_ERR_NULL;
    *out_plan = nullptr;
    if (num < 0) return COLLAGE_ERR_ARG;
    if (num > 0 && !tensors) return COLLAGE_ERR_NULL;
    if (chunk_elems == 0) chunk_elems = kDefaultChunk;
    if (chunk_elems % 2048u) return COLLAGE_ERR_ARG;

    std::vector<TensorRec> recs;
    std::vector<ChunkRec> chunks;
    std::vector<ByteRange> ranges;
    std::vector<uint64_t> first_chunk, sizes;
    std::vector<uint32_t> orig_index;
    bool has_x_lo = true, has_v_lo = true;
    uint64_t total = 0;
    for (int i = 0; i < num; ++i) {
        const collage_tensor_t& t = tensors[i];
        if (t.n == 0) continue;
        if (!t.x_hi || !t.m || !t.v_hi || !t.grad) return COLLAGE_ERR_NULL;
        if (t.n > (1ull << 62)) return COLLAGE_ERR_ARG;
        has_x_lo = has_x_lo && t.x_lo;
        has_v_lo = has_v_lo && t.v_lo;
        TensorRec r{};
        r.x_hi = static_cast<uint16_t*>(t.x_hi);
        r.x_lo = static_cast<uint16_t*>(t.x_lo);
        r.m = static_cast<uint16_t*>(t.m);
        r.v_hi = static_cast<uint16_t*>(t.v_hi);
        r.v_lo = static_cast<uint16_t*>(t.v_lo);
        r.grad = static_cast<const uint16_t*>(t.grad);
        r.n = t.n;
        r.aligned = aligned16(t.x_hi) && aligned16(t.x_lo) && aligned16(t.m) && aligned16(t.v_hi) &&
                    aligned16(t.v_lo) && aligned16(t.grad);
        for (const void* q : {static_cast<const void*>(t.x_hi), static_cast<const void*>(t.x_lo),
                              static_cast<const void*>(t.m), static_cast<const void*>(t.v_hi),
                              static_cast<const void*>(t.v_lo), t.grad})
            push_range(ranges, q, t.n);
        const uint64_t nchunks = (t.n + chunk_elems - 1) / chunk_elems;
        if (nchunks > 0xFFFFFFFFull || chunks.size() + nchunks > 0xFFFFFFFFull) return COLLAGE_ERR_ARG;
        const uint32_t id = static_cast<uint32_t>(recs.size());
        first_chunk.push_back(chunks.size());
        sizes.push_back(t.n);
        orig_index.push_back(static_cast<uint32_t>(i));
        for (uint64_t c = 0; c < nchunks; ++c) chunks.push_back({id, static_cast<uint32_t>(c)});
        recs.push_back(r);
        total += t.n;
    }
    if (any_overlap(ranges)) return COLLAGE_ERR_ALIAS;     // leaves `ranges` sorted by address
    first_chunk.push_back(chunks.size());

    collage_plan* plan = new collage_plan;
    plan->num_given = num;
    plan->ranges = ranges;
    plan->own_ranges = ranges;
    plan->given.assign(tensors, tensors + num);
    plan->num_chunks = chunks.size();
    plan->num_elements = total;
    plan->chunk_elems = chunk_elems;
    plan->num_tensors = static_cast<int>(recs.size());
    plan->has_x_lo = has_x_lo;
    plan->has_v_lo = has_v_lo;
    if (!recs.empty()) {
        if (cudaGetDevice(&plan->device) != cudaSuccess ||
            cudaMalloc(&plan->d_tensors, recs.size() * sizeof(TensorRec)) != cudaSuccess ||
            cudaMalloc(&plan->d_chunks, chunks.size() * sizeof(ChunkRec)) != cudaSuccess ||
            cudaMemcpy(plan->d_tensors, recs.data(), recs.size() * sizeof(TensorRec), cudaMemcpyHostToDevice) !=
                cudaSuccess ||
            cudaMemcpy(plan->d_chunks, chunks.data(), chunks.size() * sizeof(ChunkRec), cudaMemcpyHostToDevice) !=
                cudaSuccess ||
            cudaMalloc(&plan->d_first_chunk, first_chunk.size() * sizeof(uint64_t)) != cudaSuccess ||
            cudaMalloc(&plan->d_sizes, sizes.size() * sizeof(uint64_t)) != cudaSuccess ||
            cudaMalloc(&plan->d_orig_index, orig_index.size() * sizeof(uint32_t)) != cudaSuccess ||
            cudaMemcpy(plan->d_first_chunk, first_chunk.data(), first_chunk.size() * sizeof(uint64_t),
                       cudaMemcpyHostToDevice) != cudaSuccess ||
            cudaMemcpy(plan->d_sizes, sizes.data(), sizes.size() * sizeof(uint64_t), cudaMemcpyHostToDevice) !=
                cudaSuccess ||
            cudaMemcpy(plan->d_orig_index, orig_index.data(), orig_index.size() * sizeof(uint32_t),
                       cudaMemcpyHostToDevice) != cudaSuccess) {
            cudaFree(plan->d_tensors);
            cudaFree(plan->d_chunks);
            cudaFree(plan->d_first_chunk);
            cudaFree(plan->d_sizes);
            cudaFree(plan->d_orig_index);
            delete plan;
            return COLLAGE_ERR_CUDA;
        }
    }
    *out_plan = plan;
    return COLLAGE_OK;
}

collage_status_t collage_adamw_step_multi(const collage_plan_t* plan, const collage_hyper_t* hyper, uint64_t step,
                                          collage_strategy_t strategy, void* stream) {
    if (!plan) return COLLAGE_ERR_NULL;
    collage_status_t st = check_common(hyper, step, strategy);
    if (st != COLLAGE_OK) return st;
    if (strategy >= COLLAGE_LIGHT && !plan->has_x_lo) return COLLAGE_ERR_NULL;
    if (stores_v_lo(strategy) && !plan->has_v_lo) return COLLAGE_ERR_NULL;
    DeviceInfo dev;
    st = current_device(&dev);
    if (st != COLLAGE_OK) return st;
    if (!plan_on_current_device(plan)) return COLLAGE_ERR_ARG;
    const bool edq = hyper->edq_out != nullptr;
    if (edq) {
        // the record and the workspace may touch neither an array of the plan nor each other
        std::vector<ByteRange> own;
        push_edq_ranges(own, hyper);
        if (any_overlap(own) || overlaps_sorted(plan->ranges, hyper->edq_out, sizeof(collage_edq_t)) ||
            overlaps_sorted(plan->ranges, hyper->workspace, kWorkspaceBytes))
            return COLLAGE_ERR_ALIAS;
    }
    cudaStream_t cs = static_cast<cudaStream_t>(stream);

    StepParams p{};
    st = make_scalars(hyper, step, &p.k);
    if (st != COLLAGE_OK) return st;
    p.tensors = plan->d_tensors;
    p.chunks = plan->d_chunks;
    p.num_chunks = plan->num_chunks;
    p.chunk_elems = plan->chunk_elems;
    p.fin = make_finish(hyper->workspace, hyper->edq_out, plan->num_elements, false);
    p.replica_bases = plan->d_replica_bases;
    p.num_replicas = plan->num_replicas;
    p.num_plan_tensors = plan->num_tensors;
    int grid = 0;
    if (plan->num_chunks > 0) {
        // large tiles need chunks that are whole numbers of them (the default chunk is three)
        const bool large = plan->chunk_elems % pipe_tile(COLLAGE_PLUS, true) == 0 &&
                           takes_large_tiles(strategy, p.k.flags, hyper->flags, plan->num_elements);
        if (dispatch_step<false>(p, strategy, edq, dev.sm_count, cs, &grid, large) != cudaSuccess) return COLLAGE_ERR_CUDA;
    }
    if (edq && grid == 0) {        // an empty plan: the record still has to say so
        launch_edq_finalize(p.fin.partials, 0, 0, p.fin.out, cs, false);
        if (cudaGetLastError() != cudaSuccess) return COLLAGE_ERR_CUDA;
    }
    return COLLAGE_OK;
}

collage_status_t collage_plan_set_replicas(collage_plan_t* plan, const void* const* replicas, int num_replicas) {
    if (!plan) return COLLAGE_ERR_NULL;
    if (num_replicas < 0 || num_replicas > 15) return COLLAGE_ERR_ARG;
    if (num_replicas > 0 && !replicas) return COLLAGE_ERR_NULL;
    if (!plan_on_current_device(plan)) return COLLAGE_ERR_ARG;
    std::vector<uint64_t> bases;
    std::vector<ByteRange> ranges = plan->own_ranges;
    for (int r = 0; r < num_replicas; ++r) {
        for (int i = 0; i < plan->num_given; ++i) {
            const collage_tensor_t& t = plan->given[i];
            if (t.n == 0) continue;
            const void* q = replicas[static_cast<size_t>(r) * plan->num_given + i];
            if (!q) return COLLAGE_ERR_NULL;
            // a replica must sit like its tensor relative to 16-byte boundaries: tiles are copied whole
            if ((reinterpret_cast<uintptr_t>(q) & 15u) != (reinterpret_cast<uintptr_t>(t.x_hi) & 15u)) return COLLAGE_ERR_ARG;
            push_range(ranges, q, t.n);
            bases.push_back(reinterpret_cast<uint64_t>(q));
        }
    }
    if (any_overlap(ranges)) return COLLAGE_ERR_ALIAS;
    uint64_t* d = nullptr;
    if (!bases.empty()) {
        if (cudaMalloc(&d, bases.size() * sizeof(uint64_t)) != cudaSuccess) return COLLAGE_ERR_CUDA;
        if (cudaMemcpy(d, bases.data(), bases.size() * sizeof(uint64_t), cudaMemcpyHostToDevice) != cudaSuccess) {
            cudaFree(d);
            return COLLAGE_ERR_CUDA;
        }
    }
    if (cudaDeviceSynchronize() != cudaSuccess) return COLLAGE_ERR_CUDA;   // no step may still read the old table
    cudaFree(plan->d_replica_bases);
    plan->d_replica_bases = d;
    plan->num_replicas = bases.empty() ? 0 : num_replicas;
    plan->ranges = ranges;                 // sorted by any_overlap: later calls check their workspace against the replicas too
    return COLLAGE_OK;
}

collage_status_t collage_enable_peer_access(int peer_device) {
    int device = -1, can = 0;
    if (cudaGetDevice(&device) != cudaSuccess) return COLLAGE_ERR_CUDA;
    if (peer_device == device || peer_device < 0) return COLLAGE_ERR_ARG;
    if (cudaDeviceCanAccessPeer(&can, device, peer_device) != cudaSuccess) {
        (void)cudaGetLastError();
        return COLLAGE_ERR_ARG;
    }
    if (!can) return COLLAGE_ERR_ARG;
    const cudaError_t e = cudaDeviceEnablePeerAccess(peer_device, 0);
    if (e == cudaErrorPeerAccessAlreadyEnabled) {
        (void)cudaGetLastError();          // not an error: clear the runtime's last-error slot
        return COLLAGE_OK;
    }
    return e == cudaSuccess ? COLLAGE_OK : COLLAGE_ERR_CUDA;
}

size_t collage_plan_workspace_bytes(const collage_plan_t* plan) {
    return plan ? static_cast<size_t>(plan->num_chunks) * sizeof(EdqPartial) + sizeof(EdqPartial) : 0;
}

collage_status_t collage_adamw_step_multi_per_tensor(const collage_plan_t* plan, const collage_hyper_t* hyper,
                                                     uint64_t step, collage_strategy_t strategy,
                                                     collage_edq_t* per_tensor_out_dev, int num,
                                                     void* chunk_workspace, size_t chunk_workspace_bytes,
                                                     void* stream) {
    if (!plan || !hyper || !per_tensor_out_dev) return COLLAGE_ERR_NULL;
    collage_hyper_t h = *hyper;
    void* global_out = h.edq_out;
    h.edq_out = nullptr;                      // the block-partial workspace of the plain multi step is not used
    collage_status_t st = check_common(&h, step, strategy);
    if (st != COLLAGE_OK) return st;
    if (num != plan->num_given) return COLLAGE_ERR_ARG;
    if (h.flags & (COLLAGE_FLAG_TWOSUM_GROW | COLLAGE_FLAG_DECAY_BY_GROW)) return COLLAGE_ERR_ARG;   // not built
    if (strategy >= COLLAGE_LIGHT && !plan->has_x_lo) return COLLAGE_ERR_NULL;
    if (stores_v_lo(strategy) && !plan->has_v_lo) return COLLAGE_ERR_NULL;
    if (!chunk_workspace || (reinterpret_cast<uintptr_t>(chunk_workspace) & 15u) ||
        chunk_workspace_bytes < collage_plan_workspace_bytes(plan))
        return COLLAGE_ERR_WORKSPACE;
    DeviceInfo dev;
    st = current_device(&dev);
    if (st != COLLAGE_OK) return st;
    if (!plan_on_current_device(plan)) return COLLAGE_ERR_ARG;
    {
        // the per-tensor records, the chunk workspace and the optional total may touch neither an array
        // of the plan nor each other
        std::vector<ByteRange> own;
        push_bytes(own, per_tensor_out_dev, static_cast<uint64_t>(num) * sizeof(collage_edq_t));
        push_bytes(own, chunk_workspace, collage_plan_workspace_bytes(plan));
        push_bytes(own, global_out, sizeof(collage_edq_t));
        const std::vector<ByteRange> mine = own;
        if (any_overlap(own)) return COLLAGE_ERR_ALIAS;
        for (const ByteRange& r : mine)
            if (overlaps_sorted(plan->ranges, reinterpret_cast<const void*>(r.begin), r.end - r.begin)) return COLLAGE_ERR_ALIAS;
    }
    cudaStream_t cs = static_cast<cudaStream_t>(stream);

    StepParams p{};
    st = make_scalars(&h, step, &p.k);
    if (st != COLLAGE_OK) return st;
    p.tensors = plan->d_tensors;
    p.chunks = plan->d_chunks;
    p.num_chunks = plan->num_chunks;
    p.chunk_elems = plan->chunk_elems;
    p.chunk_partials = static_cast<EdqPartial*>(chunk_workspace);
    p.replica_bases = plan->d_replica_bases;
    p.num_replicas = plan->num_replicas;
    p.num_plan_tensors = plan->num_tensors;
    if (num > 0 && cudaMemsetAsync(per_tensor_out_dev, 0, static_cast<size_t>(num) * sizeof(collage_edq_t), cs) != cudaSuccess)
        return COLLAGE_ERR_CUDA;
    if (plan->num_chunks > 0) {
        int grid = 0;
        const bool large = plan->chunk_elems % pipe_tile(COLLAGE_PLUS, true) == 0 &&
                           takes_large_tiles(strategy, p.k.flags, h.flags, plan->num_elements);
        if (dispatch_step_per_chunk(p, strategy, dev.sm_count, cs, &grid, large) != cudaSuccess) return COLLAGE_ERR_CUDA;
        edq_per_tensor_kernel<<<plan->num_tensors, 256, 0, cs>>>(p.chunk_partials, plan->d_first_chunk, plan->d_orig_index,
                                                                 plan->d_sizes, per_tensor_out_dev);
        if (cudaGetLastError() != cudaSuccess) return COLLAGE_ERR_CUDA;
    }
    if (global_out) {
        edq_sum_records_kernel<<<1, 32, 0, cs>>>(per_tensor_out_dev, num, static_cast<collage_edq_t*>(global_out));
        if (cudaGetLastError() != cudaSuccess) return COLLAGE_ERR_CUDA;
    }
    return COLLAGE_OK;
}

collage_status_t collage_plan_destroy(collage_plan_t* plan) {
    if (!plan) return COLLAGE_OK;
    bool ok = cudaFree(plan->d_tensors) == cudaSuccess;
    ok = (cudaFree(plan->d_chunks) == cudaSuccess) && ok;
    ok = (cudaFree(plan->d_first_chunk) == cudaSuccess) && ok;
    ok = (cudaFree(plan->d_sizes) == cudaSuccess) && ok;
    ok = (cudaFree(plan->d_orig_index) == cudaSuccess) && ok;
    ok = (cudaFree(plan->d_replica_bases) == cudaSuccess) && ok;
    delete plan;
    return ok ? COLLAGE_OK : COLLAGE_ERR_CUDA;
}

uint64_t collage_plan_num_elements(const collage_plan_t* plan) { return plan ? plan->num_elements : 0; }
uint64_t collage_plan_num_chunks(const collage_plan_t* plan) { return plan ? plan->num_chunks : 0; }

collage_status_t collage_pipeline_fault(uint32_t* out_host) {
    if (!out_host) return COLLAGE_ERR_NULL;
    unsigned int v = 0, v32 = 0, zero = 0;
    if (cudaMemcpyFromSymbol(&v, g_pipeline_fault, sizeof v) != cudaSuccess) return COLLAGE_ERR_CUDA;
    if (v && cudaMemcpyToSymbol(g_pipeline_fault, &zero, sizeof zero) != cudaSuccess) return COLLAGE_ERR_CUDA;
    if (read_clear_fault32(&v32) != cudaSuccess) return COLLAGE_ERR_CUDA;    // the float comparator's pipeline
    *out_host = v ? v : v32;
    return COLLAGE_OK;
}

// ---- the give-up path of the bounded waits, exercised without a fault ---------------------------
namespace collage {
// One warp waits on a barrier that nothing completes, with a short bound; the wait runs out, the
// code 100 goes to the fault word and the kernel returns in the ordinary way.
__global__ void __launch_bounds__(32) wait_timeout_kernel(unsigned long long limit_ns) {
    __shared__ alignas(8) uint64_t bar;
    if (threadIdx.x == 0) {
        pipe::mbar_init(&bar, 1);
        pipe::mbar_init_fence();
    }
    __syncwarp();
    (void)__all_sync(0xFFFFFFFFu, pipe::mbar_wait(&bar, 0u, 99u, &g_pipeline_fault, limit_ns));
}
}  // namespace collage

collage_status_t collage_wait_timeout_selftest(uint32_t limit_ms, void* stream) {
    if (limit_ms == 0 || limit_ms > 1000) return COLLAGE_ERR_ARG;
    DeviceInfo dev;
    const collage_status_t st = current_device(&dev);
    if (st != COLLAGE_OK) return st;
    wait_timeout_kernel<<<1, 32, 0, static_cast<cudaStream_t>(stream)>>>(static_cast<unsigned long long>(limit_ms) * 1000000ULL);
    return cudaGetLastError() == cudaSuccess ? COLLAGE_OK : COLLAGE_ERR_CUDA;
}

// ---- state in host memory: staged step -------------------------------------------------------

namespace {
struct HostStepContext {
    cudaStream_t in = nullptr, out = nullptr;
    cudaEvent_t start = nullptr, loaded[2] = {nullptr, nullptr}, computed[2] = {nullptr, nullptr},
                drained[2] = {nullptr, nullptr};
    bool ready = false;
};

// Two copy streams and a handful of events per device, created on the first staged call (under a
// lock: two host threads may make that call together).
cudaError_t host_step_context(int device, HostStepContext** out) {
    static HostStepContext ctx[64];
    static std::mutex guard;
    if (device < 0 || device >= 64) return cudaErrorInvalidDevice;
    std::lock_guard<std::mutex> hold(guard);
    HostStepContext& c = ctx[device];
    if (!c.ready) {
        cudaError_t e;
        if ((e = cudaStreamCreateWithFlags(&c.in, cudaStreamNonBlocking)) != cudaSuccess) return e;
        if ((e = cudaStreamCreateWithFlags(&c.out, cudaStreamNonBlocking)) != cudaSuccess) return e;
        cudaEvent_t* evs[] = {&c.start, &c.loaded[0], &c.loaded[1], &c.computed[0], &c.computed[1], &c.drained[0],
                              &c.drained[1]};
        for (cudaEvent_t* ev : evs)
            if ((e = cudaEventCreateWithFlags(ev, cudaEventDisableTiming)) != cudaSuccess) return e;
        c.ready = true;
    }
    *out = &c;
    return cudaSuccess;
}
}  // namespace

collage_status_t collage_adamw_step_host(void* x_hi, void* x_lo, void* m, void* v_hi, void* v_lo, const void* grad,
                                         uint64_t n, const collage_hyper_t* hyper, uint64_t step,
                                         collage_strategy_t strategy, void* staging_dev, size_t staging_bytes,
                                         void* stream) {
    if (!hyper) return COLLAGE_ERR_NULL;
    collage_hyper_t h = *hyper;
    void* edq_host = h.edq_out;
    h.edq_out = nullptr;                       // workspace fields of the caller's struct are not used here
    collage_status_t st = check_common(&h, step, strategy);
    if (st != COLLAGE_OK) return st;
    if (!x_hi || !m || !v_hi || !grad) return COLLAGE_ERR_NULL;
    if ((strategy >= COLLAGE_LIGHT) != (x_lo != nullptr)) return x_lo ? COLLAGE_ERR_ARG : COLLAGE_ERR_NULL;
    if (stores_v_lo(strategy) != (v_lo != nullptr)) return v_lo ? COLLAGE_ERR_ARG : COLLAGE_ERR_NULL;
    if (n > (1ull << 62)) return COLLAGE_ERR_ARG;
    std::vector<ByteRange> ranges;
    for (const void* q : {static_cast<const void*>(x_hi), static_cast<const void*>(x_lo), static_cast<const void*>(m),
                          static_cast<const void*>(v_hi), static_cast<const void*>(v_lo), grad})
        push_range(ranges, q, n);
    if (any_overlap(ranges)) return COLLAGE_ERR_ALIAS;

    // staging layout: [record 256 B][EDQ workspace][2 slabs x 6 arrays x slab_elems bfloat16]
    const size_t fixed = 256 + kWorkspaceBytes;
    if (!staging_dev || (reinterpret_cast<uintptr_t>(staging_dev) & 255u) || staging_bytes < fixed + 2 * 6 * 2 * 16384)
        return COLLAGE_ERR_WORKSPACE;
    const uint64_t slab = (staging_bytes - fixed) / (2 * 6 * 2) / 16384 * 16384;
    DeviceInfo dev;
    st = current_device(&dev);
    if (st != COLLAGE_OK) return st;
    int device = 0;
    HostStepContext* c = nullptr;
    if (cudaGetDevice(&device) != cudaSuccess || host_step_context(device, &c) != cudaSuccess) return COLLAGE_ERR_CUDA;
    cudaStream_t cs = static_cast<cudaStream_t>(stream);
    StepScalars k;
    st = make_scalars(&h, step, &k);
    if (st != COLLAGE_OK) return st;

    char* base = static_cast<char*>(staging_dev);
    collage_edq_t* record = reinterpret_cast<collage_edq_t*>(base);
    EdqPartial* partials = reinterpret_cast<EdqPartial*>(base + 256);
    uint16_t* slabs = reinterpret_cast<uint16_t*>(base + fixed);
    auto dev_array = [&](int buf, int a) { return slabs + (static_cast<uint64_t>(buf) * 6 + a) * slab; };
    uint16_t* host_rw[5] = {static_cast<uint16_t*>(x_hi), static_cast<uint16_t*>(x_lo), static_cast<uint16_t*>(m),
                            static_cast<uint16_t*>(v_hi), static_cast<uint16_t*>(v_lo)};
    const uint16_t* host_g = static_cast<const uint16_t*>(grad);
    const bool edq = edq_host != nullptr;
#define COLLAGE_TRY(call) do { if ((call) != cudaSuccess) return COLLAGE_ERR_CUDA; } while (0)

    if (edq) {
        COLLAGE_TRY(cudaMemsetAsync(record, 0, sizeof(collage_edq_t), cs));
        COLLAGE_TRY(cudaMemsetAsync(reinterpret_cast<char*>(partials) + kTicketOffset, 0, 64, cs));   // the staging buffer is ours to clear
    }
    COLLAGE_TRY(cudaEventRecord(c->start, cs));               // copies start after the caller's earlier work
    COLLAGE_TRY(cudaStreamWaitEvent(c->in, c->start, 0));
    const uint64_t nslabs = (n + slab - 1) / slab;
    for (uint64_t i = 0; i < nslabs; ++i) {
        const int b = static_cast<int>(i & 1);
        const uint64_t off = i * slab, len = (n - off < slab) ? n - off : slab;
        if (i >= 2) COLLAGE_TRY(cudaStreamWaitEvent(c->in, c->drained[b], 0));   // slab i-2 has left buffer b
        for (int a = 0; a < 5; ++a)
            if (host_rw[a])
                COLLAGE_TRY(cudaMemcpyAsync(dev_array(b, a), host_rw[a] + off, 2 * len, cudaMemcpyHostToDevice, c->in));
        COLLAGE_TRY(cudaMemcpyAsync(dev_array(b, 5), host_g + off, 2 * len, cudaMemcpyHostToDevice, c->in));
        COLLAGE_TRY(cudaEventRecord(c->loaded[b], c->in));
        COLLAGE_TRY(cudaStreamWaitEvent(cs, c->loaded[b], 0));
        int grid = 0;
        COLLAGE_TRY(launch_flat(dev_array(b, 0), x_lo ? dev_array(b, 1) : nullptr, dev_array(b, 2), dev_array(b, 3),
                                v_lo ? dev_array(b, 4) : nullptr, dev_array(b, 5), len, k, strategy,
                                make_finish(partials, edq ? record : nullptr, len, true), dev.sm_count, cs, &grid, h.flags));
        COLLAGE_TRY(cudaEventRecord(c->computed[b], cs));
        COLLAGE_TRY(cudaStreamWaitEvent(c->out, c->computed[b], 0));
        for (int a = 0; a < 5; ++a)
            if (host_rw[a])
                COLLAGE_TRY(cudaMemcpyAsync(host_rw[a] + off, dev_array(b, a), 2 * len, cudaMemcpyDeviceToHost, c->out));
        COLLAGE_TRY(cudaEventRecord(c->drained[b], c->out));
    }
    for (uint64_t i = (nslabs >= 2 ? nslabs - 2 : 0); i < nslabs; ++i)
        COLLAGE_TRY(cudaStreamWaitEvent(cs, c->drained[i & 1], 0));              // results are home before `stream` goes on
    if (edq) COLLAGE_TRY(cudaMemcpyAsync(edq_host, record, sizeof(collage_edq_t), cudaMemcpyDeviceToHost, cs));
#undef COLLAGE_TRY
    return COLLAGE_OK;
}

}  // extern "C"
