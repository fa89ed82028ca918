// Comparator step: option D of the paper's Table 2 (bfloat16 parameter and gradient, float
// optimizer states, float master weights) and D^-MW (Section 5.1: the same without master weights).
// Standard mixed-precision AdamW, every operation one IEEE single-precision operation in the order
// of Algorithm 2, scalars evaluated in double on the host and cast to float once.
//
// Same data movement as the bfloat16 step: a producer thread bulk-copies tiles of every array into
// shared memory (cp.async.bulk + mbarrier, three stages), 512 consumers compute and write back, the
// producer bulk-stores.  Traffic per parameter: D 28 B (reads g 2, m 4, v 4, w 4; writes theta 2,
// m 4, v 4, w 4), D^-MW 22 B.
#include "bulk_pipe.cuh"
#include "host_common.cuh"
#include "edq_reduce.cuh"
#include "mcf_device.cuh"

namespace collage {

void launch_edq_finalize(const EdqPartial* partials, int count, uint64_t n, collage_edq_t* out, cudaStream_t stream,
                         bool accumulate);
// fault word of this translation unit's pipeline (device symbols are not shared across units);
// collage_pipeline_fault reports it together with the bfloat16 step's
static __device__ unsigned int g_pipeline_fault32 = 0;


struct Fp32Scalars {
    float b1, c1, b2, c2, bc1, bc2, neg_a, lam, eps;
    uint32_t flags;
};

struct Fp32Params {
    uint16_t* theta;
    float* master;        // nullptr: no master weights
    float* m;
    float* v;
    const uint16_t* grad;
    uint64_t n;
    int aligned;          // every pointer is 16-byte aligned
    Fp32Scalars k;
    EdqFinish fin;              // per-block partials, ticket and record of the EDQ reduction
};

// Geometry of the pipeline (one block per SM, a producer warp beside the consumers).  The version
// without master weights moves 22 B per parameter for the same IEEE divisions and root as the
// 28 B one, so its arithmetic weighs more and it wants more consumer threads: measured on a flat
// 2^30 tensor, 512 / 768 / 960 consumers gave 5.2 / 5.7 / 5.9 TB/s without master weights and
// 6.3 / 6.4 / 6.3 TB/s with them.
#ifndef COLLAGE_FP32_CONSUMERS
#define COLLAGE_FP32_CONSUMERS 768
#endif
#ifndef COLLAGE_FP32_CONSUMERS_NO_MASTER
#define COLLAGE_FP32_CONSUMERS_NO_MASTER 960
#endif
#ifndef COLLAGE_FP32_QUADS
#define COLLAGE_FP32_QUADS 1
#endif
#ifndef COLLAGE_FP32_STAGES
#define COLLAGE_FP32_STAGES 3
#endif
template <bool MASTER>
struct Fp32Geometry {
    static constexpr int kCons = MASTER ? COLLAGE_FP32_CONSUMERS : COLLAGE_FP32_CONSUMERS_NO_MASTER;   // consumer threads
    static constexpr int kQuads = COLLAGE_FP32_QUADS;      // groups of 4 consecutive elements per thread and tile
    static constexpr int kTile = kCons * 4 * kQuads;       // elements per tile
    static constexpr int kStages = COLLAGE_FP32_STAGES;
};

template <bool MASTER>
struct Fp32Stage {
    static constexpr int kTile = Fp32Geometry<MASTER>::kTile;
    alignas(128) float m[kTile];
    alignas(128) float v[kTile];
    alignas(128) float w[MASTER ? kTile : 32];
    alignas(128) uint16_t theta[kTile];
    alignas(128) uint16_t g[kTile];
};
template <bool MASTER>
struct Fp32Smem {
    static constexpr int kStages = Fp32Geometry<MASTER>::kStages, kCons = Fp32Geometry<MASTER>::kCons;
    Fp32Stage<MASTER> stage[kStages];
    alignas(8) uint64_t full[kStages];
    alignas(8) uint64_t done[kStages];
    double red_dot[kCons / 32], red_sq[kCons / 32];
    unsigned long long red_lost[kCons / 32];
    EdqFinishSmem finish;
};

// One parameter: Algorithm 2 lines 8-13 in float.  Returns the update; w is the stored float
// parameter (master weight, or the widened bfloat16 parameter), updated in place.
__device__ __forceinline__ float adamw_fp32_element(float& m, float& v, float& w, float g, const Fp32Scalars& k) {
    m = __fadd_rn(__fmul_rn(k.b1, m), __fmul_rn(k.c1, g));
    v = __fadd_rn(__fmul_rn(k.b2, v), __fmul_rn(k.c2, __fmul_rn(g, g)));
    const float mhat = __fdiv_rn(m, k.bc1);
    const float vhat = __fdiv_rn(v, k.bc2);
    const float den = (k.flags & 1u) ? __fsqrt_rn(__fadd_rn(vhat, k.eps)) : __fadd_rn(__fsqrt_rn(vhat), k.eps);
    const float u = __fadd_rn(__fdiv_rn(mhat, den), __fmul_rn(k.lam, w));
    const float delta = __fmul_rn(k.neg_a, u);
    w = __fadd_rn(w, delta);
    return delta;
}

__device__ __forceinline__ uint16_t to_bf16_rn(float x) {
    uint16_t h;
    asm("cvt.rn.bf16.f32 %0, %1;" : "=h"(h) : "f"(x));
    return h;
}
__device__ __forceinline__ float from_bf16(uint16_t h) { return __uint_as_float(static_cast<uint32_t>(h) << 16); }

struct Fp32Acc {
    float dot, sq;
    uint32_t lost;
};

// element step plus its EDQ terms; `theta` in/out is the bfloat16 parameter
template <bool MASTER, bool EDQ>
__device__ __forceinline__ void fp32_element(float& m, float& v, float& w, uint16_t& theta, float g, const Fp32Scalars& k,
                                             Fp32Acc& acc) {
    float stored = MASTER ? w : from_bf16(theta);
    const float before = stored;
    const float delta = adamw_fp32_element(m, v, stored, g, k);
    const uint16_t theta_new = to_bf16_rn(stored);
    if (EDQ) {
        // effective update of the stored parameter: the master weight, or the bfloat16 parameter
        const float after = MASTER ? stored : from_bf16(theta_new);
        const float eff = __fsub_rn(after, before);
        acc.dot = __fadd_rn(acc.dot, __fmul_rn(delta, eff));
        acc.sq = __fadd_rn(acc.sq, __fmul_rn(delta, delta));
        acc.lost += (delta != 0.0f && after == before) ? 1u : 0u;
    }
    if (MASTER) w = stored;
    theta = theta_new;
}

template <bool MASTER, bool EDQ>
__global__ void __launch_bounds__(Fp32Geometry<MASTER>::kCons + 32, 1) adamw_fp32_pipeline_kernel(const __grid_constant__ Fp32Params p) {
    constexpr int kCons32 = Fp32Geometry<MASTER>::kCons, kQuads32 = Fp32Geometry<MASTER>::kQuads;
    constexpr int kTile32 = Fp32Geometry<MASTER>::kTile, kStages32 = Fp32Geometry<MASTER>::kStages;
    extern __shared__ unsigned char smem_raw[];
    Fp32Smem<MASTER>& sm = *reinterpret_cast<Fp32Smem<MASTER>*>((reinterpret_cast<uintptr_t>(smem_raw) + 127) & ~static_cast<uintptr_t>(127));
    constexpr int kWarps = kCons32 / 32;
    const bool is_producer = threadIdx.x >= kCons32;
    if (threadIdx.x == 0) {
#pragma unroll
        for (int s = 0; s < kStages32; ++s) {
            pipe::mbar_init(&sm.full[s], 1);
            pipe::mbar_init(&sm.done[s], kWarps);
        }
        pipe::mbar_init_fence();
    }
    __syncthreads();

    const uint64_t num_tiles = (p.n + kTile32 - 1) / kTile32;
    const Fp32Scalars& k = p.k;
    double dot = 0.0, sq = 0.0;
    uint32_t lost = 0;
    uint32_t it = 0;
    bool alive = true;

    if (is_producer) {
        if (threadIdx.x == kCons32) {
            uint64_t held[kStages32];          // tile number sitting in each stage
            bool held_bulk[kStages32];
#pragma unroll
            for (int s = 0; s < kStages32; ++s) {
                held[s] = 0;
                held_bulk[s] = false;
            }
            auto store_out = [&](int s) {
                const uint64_t off = held[s] * kTile32;
                pipe::bulk_store(p.theta + off, sm.stage[s].theta, kTile32 * 2);
                pipe::bulk_store(p.m + off, sm.stage[s].m, kTile32 * 4);
                pipe::bulk_store(p.v + off, sm.stage[s].v, kTile32 * 4);
                if (MASTER) pipe::bulk_store(p.master + off, sm.stage[s].w, kTile32 * 4);
                pipe::bulk_commit();
            };
            for (uint64_t tile = blockIdx.x; tile < num_tiles && alive; tile += gridDim.x, ++it) {
                const int s = it % kStages32;
                const uint32_t use = it / kStages32;
                if (use > 0) {
                    alive = pipe::mbar_wait(&sm.done[s], (use - 1) & 1u, 60u + s, &g_pipeline_fault32);
                    if (!alive) break;
                    if (held_bulk[s]) {
                        store_out(s);
                        pipe::bulk_wait_read_all();
                    }
                }
                const uint64_t off = tile * kTile32;
                const bool bulk = p.aligned && (p.n - off) >= static_cast<uint64_t>(kTile32);
                held[s] = tile;
                held_bulk[s] = bulk;
                if (bulk) {
                    const uint32_t bytes = kTile32 * (2 + 4 + 4 + (MASTER ? 4 : 2));
                    pipe::mbar_arrive_expect_tx(&sm.full[s], bytes);
                    pipe::bulk_load(sm.stage[s].g, p.grad + off, kTile32 * 2, &sm.full[s]);
                    pipe::bulk_load(sm.stage[s].m, p.m + off, kTile32 * 4, &sm.full[s]);
                    pipe::bulk_load(sm.stage[s].v, p.v + off, kTile32 * 4, &sm.full[s]);
                    if (MASTER) pipe::bulk_load(sm.stage[s].w, p.master + off, kTile32 * 4, &sm.full[s]);
                    else pipe::bulk_load(sm.stage[s].theta, p.theta + off, kTile32 * 2, &sm.full[s]);
                } else {
                    pipe::mbar_arrive(&sm.full[s]);
                }
            }
            const uint32_t tail = it < static_cast<uint32_t>(kStages32) ? it : kStages32;
            for (uint32_t j = it - tail; j < it && alive; ++j) {
                const int s = j % kStages32;
                alive = pipe::mbar_wait(&sm.done[s], (j / kStages32) & 1u, 70u + s, &g_pipeline_fault32);
                if (!alive) break;
                if (held_bulk[s]) store_out(s);
            }
            if (!alive) {
                for (int s = 0; s < kStages32; ++s)
                    if (it > static_cast<uint32_t>(s)) pipe::mbar_wait(&sm.full[s], ((it - 1 - s) / kStages32) & 1u, 80u + s, &g_pipeline_fault32);
            }
            pipe::bulk_wait_all();
        }
    } else {
        const int lane = threadIdx.x & 31;
        for (uint64_t tile = blockIdx.x; tile < num_tiles; tile += gridDim.x, ++it) {
            const int s = it % kStages32;
            alive = __all_sync(0xFFFFFFFFu, pipe::mbar_wait(&sm.full[s], (it / kStages32) & 1u, 90u + s, &g_pipeline_fault32));
            if (!alive) break;
            const uint64_t off = tile * kTile32;
            Fp32Acc acc = {0.0f, 0.0f, 0u};
            if (p.aligned && (p.n - off) >= static_cast<uint64_t>(kTile32)) {
                Fp32Stage<MASTER>& st = sm.stage[s];
#pragma unroll
                for (int q = 0; q < kQuads32; ++q) {
                    const int e = (q * kCons32 + threadIdx.x) * 4;
                    float4 m4 = *reinterpret_cast<const float4*>(&st.m[e]);
                    float4 v4 = *reinterpret_cast<const float4*>(&st.v[e]);
                    float4 w4 = MASTER ? *reinterpret_cast<const float4*>(&st.w[e]) : make_float4(0.f, 0.f, 0.f, 0.f);
                    const uint2 g2 = *reinterpret_cast<const uint2*>(&st.g[e]);
                    uint2 t2 = MASTER ? make_uint2(0u, 0u) : *reinterpret_cast<const uint2*>(&st.theta[e]);
                    float* mm = reinterpret_cast<float*>(&m4);
                    float* vv = reinterpret_cast<float*>(&v4);
                    float* ww = reinterpret_cast<float*>(&w4);
                    const uint32_t gw[2] = {g2.x, g2.y};
                    uint32_t tw[2] = {t2.x, t2.y};
#pragma unroll
                    for (int j = 0; j < 4; ++j) {
                        uint16_t th = static_cast<uint16_t>(tw[j >> 1] >> (16 * (j & 1)));
                        const float g = from_bf16(static_cast<uint16_t>(gw[j >> 1] >> (16 * (j & 1))));
                        fp32_element<MASTER, EDQ>(mm[j], vv[j], ww[j], th, g, k, acc);
                        tw[j >> 1] = (tw[j >> 1] & ~(0xFFFFu << (16 * (j & 1)))) | (static_cast<uint32_t>(th) << (16 * (j & 1)));
                    }
                    *reinterpret_cast<float4*>(&st.m[e]) = m4;
                    *reinterpret_cast<float4*>(&st.v[e]) = v4;
                    if (MASTER) *reinterpret_cast<float4*>(&st.w[e]) = w4;
                    *reinterpret_cast<uint2*>(&st.theta[e]) = make_uint2(tw[0], tw[1]);
                }
                pipe::fence_async_smem();
            } else {
                // ragged last tile or unaligned arrays: element by element, straight from global memory
                const uint64_t end = (p.n - off) < static_cast<uint64_t>(kTile32) ? p.n : off + kTile32;
                for (uint64_t i = off + threadIdx.x; i < end; i += kCons32) {
                    float m = p.m[i], v = p.v[i], w = MASTER ? p.master[i] : 0.0f;
                    uint16_t th = p.theta[i];
                    fp32_element<MASTER, EDQ>(m, v, w, th, from_bf16(p.grad[i]), k, acc);
                    p.m[i] = m;
                    p.v[i] = v;
                    if (MASTER) p.master[i] = w;
                    p.theta[i] = th;
                }
            }
            if (EDQ) {
                dot += static_cast<double>(acc.dot);
                sq += static_cast<double>(acc.sq);
                lost += acc.lost;
            }
            __syncwarp();
            if (lane == 0) pipe::mbar_arrive(&sm.done[s]);
        }
    }

    if (EDQ) {
        unsigned long long lost64 = lost;
        if (!is_producer) {
#pragma unroll
            for (int o = 16; o > 0; o >>= 1) {
                dot += __shfl_down_sync(0xFFFFFFFFu, dot, o);
                sq += __shfl_down_sync(0xFFFFFFFFu, sq, o);
                lost64 += __shfl_down_sync(0xFFFFFFFFu, lost64, o);
            }
            if ((threadIdx.x & 31) == 0) {
                sm.red_dot[threadIdx.x >> 5] = dot;
                sm.red_sq[threadIdx.x >> 5] = sq;
                sm.red_lost[threadIdx.x >> 5] = lost64;
            }
        }
        __syncthreads();
        double d = 0.0, q = 0.0;
        unsigned long long l = 0;
        if (threadIdx.x == 0) {
#pragma unroll
            for (int w = 0; w < kWarps; ++w) {
                d += sm.red_dot[w];
                q += sm.red_sq[w];
                l += sm.red_lost[w];
            }
        }
        // one partial per block; the block that finishes last adds them up and writes the record
        edq_publish_and_finish(p.fin, sm.finish, d, q, l, &g_pipeline_fault32);
    }
}

template <bool MASTER, bool EDQ>
static cudaError_t launch_fp32(const Fp32Params& p, int sm_count, cudaStream_t stream, int* grid_out) {
    auto kernel = adamw_fp32_pipeline_kernel<MASTER, EDQ>;
    constexpr size_t smem = sizeof(Fp32Smem<MASTER>) + 128;
    constexpr int kTile32 = Fp32Geometry<MASTER>::kTile, kCons32 = Fp32Geometry<MASTER>::kCons;
    static std::atomic<bool> ready[64];     // racing first calls set the same attribute twice: harmless
    int device = 0;
    if (cudaGetDevice(&device) != cudaSuccess || device < 0 || device >= 64) return cudaErrorInvalidDevice;
    if (!ready[device].load(std::memory_order_acquire)) {
        const cudaError_t e = cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, static_cast<int>(smem));
        if (e != cudaSuccess) return e;
        ready[device].store(true, std::memory_order_release);
    }
    const uint64_t tiles = (p.n + kTile32 - 1) / kTile32;
    uint64_t grid = static_cast<uint64_t>(sm_count);
    if (grid > tiles) grid = tiles;
    *grid_out = static_cast<int>(grid);
    kernel<<<static_cast<unsigned>(grid), kCons32 + 32, smem, stream>>>(p);
    return cudaGetLastError();
}

// read and clear this unit's fault word (called by collage_pipeline_fault)
cudaError_t read_clear_fault32(unsigned int* out) {
    unsigned int v = 0, zero = 0;
    cudaError_t e = cudaMemcpyFromSymbol(&v, g_pipeline_fault32, sizeof v);
    if (e == cudaSuccess && v) e = cudaMemcpyToSymbol(g_pipeline_fault32, &zero, sizeof zero);
    *out = v;
    return e;
}

}  // namespace collage

using namespace collage;

extern "C" collage_status_t collage_adamw_step_fp32(void* theta, void* master, void* m, void* v, const void* grad,
                                                    uint64_t n, const collage_hyper_t* hyper, uint64_t step,
                                                    void* stream) {
    if (!hyper) return COLLAGE_ERR_NULL;
    if (step == 0 || !hyper_in_range(hyper)) return COLLAGE_ERR_ARG;
    if (hyper->flags & ~(COLLAGE_FLAG_EPS_INSIDE_SQRT | COLLAGE_FLAG_PIPELINE_KERNEL | COLLAGE_FLAG_DIRECT_KERNEL | COLLAGE_FLAG_LARGE_TILES))
        return COLLAGE_ERR_ARG;                               // the kernel-choice flags mean nothing here and are ignored
    if (hyper->edq_out) {
        if (!hyper->workspace || hyper->workspace_bytes < kWorkspaceBytes ||
            (reinterpret_cast<uintptr_t>(hyper->workspace) & 15u))
            return COLLAGE_ERR_WORKSPACE;
        if (reinterpret_cast<uintptr_t>(hyper->edq_out) & 7u) return COLLAGE_ERR_ARG;
    }
    if (!theta || !m || !v || !grad) return COLLAGE_ERR_NULL;
    if (n > (1ull << 61)) return COLLAGE_ERR_ARG;
    if ((reinterpret_cast<uintptr_t>(m) | reinterpret_cast<uintptr_t>(v) | reinterpret_cast<uintptr_t>(master)) & 3u)
        return COLLAGE_ERR_ARG;                               // float arrays must be 4-byte aligned
    std::vector<ByteRange> ranges;
    auto add = [&](const void* q, uint64_t bytes) {
        if (q && bytes) ranges.push_back({reinterpret_cast<uintptr_t>(q), reinterpret_cast<uintptr_t>(q) + bytes});
    };
    add(theta, 2 * n);
    add(grad, 2 * n);
    add(m, 4 * n);
    add(v, 4 * n);
    add(master, 4 * n);
    if (hyper->edq_out) {
        add(hyper->edq_out, sizeof(collage_edq_t));
        add(hyper->workspace, kWorkspaceBytes);
    }
    if (any_overlap(ranges)) return COLLAGE_ERR_ALIAS;
    DeviceInfo dev;
    const collage_status_t st = current_device(&dev);
    if (st != COLLAGE_OK) return st;

    Fp32Params p{};
    p.theta = static_cast<uint16_t*>(theta);
    p.master = static_cast<float*>(master);
    p.m = static_cast<float*>(m);
    p.v = static_cast<float*>(v);
    p.grad = static_cast<const uint16_t*>(grad);
    p.n = n;
    p.aligned = ((reinterpret_cast<uintptr_t>(theta) | reinterpret_cast<uintptr_t>(master) | reinterpret_cast<uintptr_t>(m) |
                  reinterpret_cast<uintptr_t>(v) | reinterpret_cast<uintptr_t>(grad)) & 15u) == 0;
    const double t = static_cast<double>(step);
    p.k.b1 = static_cast<float>(hyper->beta1);
    p.k.c1 = static_cast<float>(1.0 - hyper->beta1);
    p.k.b2 = static_cast<float>(hyper->beta2);
    p.k.c2 = static_cast<float>(1.0 - hyper->beta2);
    p.k.bc1 = static_cast<float>(1.0 - std::pow(hyper->beta1, t));
    p.k.bc2 = static_cast<float>(1.0 - std::pow(hyper->beta2, t));
    p.k.neg_a = -static_cast<float>(hyper->lr);
    p.k.lam = static_cast<float>(hyper->weight_decay);
    p.k.eps = static_cast<float>(hyper->eps);
    p.k.flags = hyper->flags & COLLAGE_FLAG_EPS_INSIDE_SQRT;
    if (hyper->edq_out) {
        p.fin.partials = static_cast<EdqPartial*>(hyper->workspace);
        p.fin.ticket = reinterpret_cast<unsigned int*>(static_cast<char*>(hyper->workspace) + kTicketOffset);
        p.fin.out = static_cast<collage_edq_t*>(hyper->edq_out);
        p.fin.n = n;
        p.fin.accumulate = 0;
    }
    cudaStream_t cs = static_cast<cudaStream_t>(stream);
    const bool edq = hyper->edq_out != nullptr;
    int grid = 0;
    if (n > 0) {
        cudaError_t e;
        if (master) e = edq ? launch_fp32<true, true>(p, dev.sm_count, cs, &grid) : launch_fp32<true, false>(p, dev.sm_count, cs, &grid);
        else e = edq ? launch_fp32<false, true>(p, dev.sm_count, cs, &grid) : launch_fp32<false, false>(p, dev.sm_count, cs, &grid);
        if (e != cudaSuccess) return COLLAGE_ERR_CUDA;
    }
    if (edq && grid == 0) {        // nothing was launched (n == 0): the record still has to say so
        launch_edq_finalize(p.fin.partials, 0, 0, p.fin.out, cs, false);
        if (cudaGetLastError() != cudaSuccess) return COLLAGE_ERR_CUDA;
    }
    return COLLAGE_OK;
}
