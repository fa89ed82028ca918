// The step kernel for SMALL flat tensors: no staging pipeline, one 8-parameter vector per thread
// straight from global memory, as many thread blocks in flight as the tensor has work for.
//
// The bulk-copy pipeline (step_pipeline.cuh) is built for streams much longer than the machine is
// wide: one block per SM walks tiles of 4096 or 6144 parameters.  A tensor of a few million
// parameters gives each SM one or two tiles, so most of a step is the latency of a single
// load - compute - store chain per SM.  Here every thread issues its six 16-byte loads at once and
// thousands of such threads are resident, which is the shortest chain this step admits.
// Same arithmetic (compute_vec_fast / compute_vec), same results, same EDQ reduction.
#pragma once
#include "edq_reduce.cuh"
#include "mcf_device.cuh"

namespace collage {

constexpr int kDirectThreads = 256;
// resident blocks per SM the register allocation aims for
#ifndef COLLAGE_DIRECT_MINBLOCKS
#define COLLAGE_DIRECT_MINBLOCKS 2
#endif

// A vector the lean chain gave up on: nothing has been stored yet, so its inputs are still in
// global memory.  Out of line: it runs for a vanishing share of the vectors.
template <int STRATEGY, bool EDQ, bool VARIANT>
__device__ __noinline__ VecSums careful_vector_direct(const TensorRec& t, uint64_t off, const StepScalars& k) {
    VecSums r = {0.0, 0.0, 0u};
    Vec v;
    if (t.aligned) load_vec<STRATEGY>(v, t, off);
    else load_elems<STRATEGY>(v, t, off, 8);
    compute_vec<STRATEGY, EDQ, VARIANT>(v, k, 8, r.dot, r.sq, r.lost);
    if (t.aligned) store_vec<STRATEGY>(v, t, off);
    else store_elems<STRATEGY>(v, t, off, 8);
    return r;
}

template <int STRATEGY, bool EDQ, bool FAST, bool VARIANT>
__global__ void __launch_bounds__(kDirectThreads, COLLAGE_DIRECT_MINBLOCKS) adamw_step_direct_kernel(const __grid_constant__ StepParams p) {
    __shared__ double red_dot[kDirectThreads / 32], red_sq[kDirectThreads / 32];
    __shared__ unsigned long long red_lost[kDirectThreads / 32];
    __shared__ EdqFinishSmem finish;
    const TensorRec& t = p.flat;
    const StepScalars& k = p.k;
    const uint64_t nvec = t.n >> 3;
    const int rem = static_cast<int>(t.n & 7u);
    double dot = 0.0, sq = 0.0;
    uint32_t lost = 0;
    const uint64_t stride = static_cast<uint64_t>(gridDim.x) * kDirectThreads;
    for (uint64_t i = blockIdx.x * static_cast<uint64_t>(kDirectThreads) + threadIdx.x; i < nvec; i += stride) {
        const uint64_t off = i * 8;
        Vec v;
        if (t.aligned) load_vec<STRATEGY>(v, t, off);
        else load_elems<STRATEGY>(v, t, off, 8);
        if constexpr (FAST && STRATEGY != 4) {
            if (compute_vec_fast<STRATEGY, EDQ, VARIANT>(v, k, dot, sq, lost) == 0u) {
                if (t.aligned) store_vec<STRATEGY>(v, t, off);
                else store_elems<STRATEGY>(v, t, off, 8);
            } else {
                const VecSums r = careful_vector_direct<STRATEGY, EDQ, VARIANT>(t, off, k);
                if (EDQ) {
                    dot += r.dot;
                    sq += r.sq;
                    lost += r.lost;
                }
            }
        } else {
            compute_vec<STRATEGY, EDQ, VARIANT>(v, k, 8, dot, sq, lost);
            if (t.aligned) store_vec<STRATEGY>(v, t, off);
            else store_elems<STRATEGY>(v, t, off, 8);
        }
    }
    if (rem && blockIdx.x == 0 && threadIdx.x == 0) {            // the ragged end of the tensor
        Vec v;
        load_elems<STRATEGY>(v, t, nvec * 8, rem);
        compute_vec<STRATEGY, EDQ, VARIANT>(v, k, rem, dot, sq, lost);
        store_elems<STRATEGY>(v, t, nvec * 8, rem);
    }
    if (EDQ) {
        unsigned long long lost64 = lost;
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) {
            dot += __shfl_down_sync(0xFFFFFFFFu, dot, o);
            sq += __shfl_down_sync(0xFFFFFFFFu, sq, o);
            lost64 += __shfl_down_sync(0xFFFFFFFFu, lost64, o);
        }
        if ((threadIdx.x & 31) == 0) {
            red_dot[threadIdx.x >> 5] = dot;
            red_sq[threadIdx.x >> 5] = sq;
            red_lost[threadIdx.x >> 5] = lost64;
        }
        __syncthreads();
        double d = 0.0, q = 0.0;
        unsigned long long l = 0;
        if (threadIdx.x == 0) {
#pragma unroll
            for (int w = 0; w < kDirectThreads / 32; ++w) {
                d += red_dot[w];
                q += red_sq[w];
                l += red_lost[w];
            }
        }
        edq_publish_and_finish(p.fin, finish, d, q, l, &g_pipeline_fault);
    }
}

}  // namespace collage
