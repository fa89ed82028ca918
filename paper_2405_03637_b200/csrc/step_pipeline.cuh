// The fused AdamW step kernel: a bulk-copy pipeline around the arithmetic of mcf_device.cuh.
//
// Each block walks its chunks of the chunk table (or of the one flat tensor).  One producer
// thread per block moves whole tiles (kTile elements of every state array) between
// global and shared memory with the bulk asynchronous copy engine (cp.async.bulk, completion on
// an mbarrier), kStages tiles deep, while the consumer warps compute out of shared memory and
// write their results back into the same shared slots, from where the producer bulk-stores them.
// Bytes in flight per SM no longer depend on registers or on how long the arithmetic takes.
//
//   full[s]  : producer -> consumers, "tile in stage s has landed" (1 arrival + transaction bytes)
//   done[s]  : consumers -> producer, "stage s is computed and written back" (one arrival per warp)
//
// Tiles that cannot be bulk-copied (tensor not 16-byte aligned, or the ragged last tile of a
// tensor) flow through the same barriers but are processed straight from global memory.
// Every wait is bounded: after two seconds a thread records a fault in g_pipeline_fault and leaves.
// EDQ: float within a vector, double per thread, fixed-order tree per block, one partial per block;
// the block that finishes last adds the partials (edq_reduce.cuh), so a step is one launch.
//
// On the host-validated lean chain (FAST) a consumer runs the branch-free compute_vec_fast on its
// 8 parameters; a vector with a lane that chain cannot answer is repeated in place, from the tile
// that still holds its inputs, by the out-of-line careful_vector_in_tile.
#pragma once
#include "bulk_pipe.cuh"
#include "edq_reduce.cuh"
#include "mcf_device.cuh"

namespace collage {

__device__ unsigned int g_pipeline_fault = 0;   // 0 = none; else 1 + index of the wait that gave up


// Number of state arrays read / written per option
template <int STRATEGY>
struct ArrayCount {
    static constexpr int kIn = 4 + (stores_x_lo(STRATEGY) ? 1 : 0) + (stores_v_lo(STRATEGY) ? 1 : 0);
    static constexpr int kOut = kIn - 1;   // everything but the gradient
};

// order of the arrays inside a stage: th, m, v, [dth], [dv], g  (outputs first, gradient last)
template <int STRATEGY>
__device__ __forceinline__ void tile_pointers(const TensorRec& t, uint64_t off, uint16_t* (&out)[5], const uint16_t*& g) {
    int a = 0;
    out[a++] = t.x_hi + off;
    out[a++] = t.m + off;
    out[a++] = t.v_hi + off;
    if (stores_x_lo(STRATEGY)) out[a++] = t.x_lo + off;
    if (stores_v_lo(STRATEGY)) out[a++] = t.v_lo + off;
    g = t.grad + off;
}

// address of element `elem` of tensor `tensor` in replica r (a plan-wide table of base addresses)
__device__ __forceinline__ uint16_t* replica_ptr(const StepParams& p, int r, uint32_t tensor, uint64_t elem) {
    return reinterpret_cast<uint16_t*>(p.replica_bases[static_cast<uint64_t>(r) * p.num_plan_tensors + tensor]) + elem;
}

template <int CONSUMERS, int VPT, int STAGES, int STRATEGY>
struct PipeSmem {
    static constexpr int kTile = CONSUMERS * 8 * VPT;
    alignas(128) uint16_t data[STAGES][ArrayCount<STRATEGY>::kIn][kTile];
    alignas(8) uint64_t full[STAGES];
    alignas(8) uint64_t done[STAGES];
    alignas(8) uint64_t red_full, red_free;   // hand-over of per-chunk EDQ sums (PER_CHUNK only)
    double red_dot[CONSUMERS / 32], red_sq[CONSUMERS / 32];
    unsigned long long red_lost[CONSUMERS / 32];
    EdqFinishSmem finish;                     // the last block's sum over all blocks (EDQ, not PER_CHUNK)
};

// PER_CHUNK: the EDQ sums are written once per chunk (p.chunk_partials[chunk]) instead of once per
// block, so that a later kernel can add them up tensor by tensor.
template <int STRATEGY, bool EDQ, bool FLAT, bool FAST, int CONSUMERS, int VPT, int STAGES, bool PER_CHUNK = false,
          bool VARIANT = false>
__global__ void __launch_bounds__(CONSUMERS + 32, COLLAGE_PIPE_MINBLOCKS)
adamw_step_pipeline_kernel(const __grid_constant__ StepParams p) {
    constexpr int kTile = CONSUMERS * 8 * VPT;
    constexpr int NIN = ArrayCount<STRATEGY>::kIn, NOUT = ArrayCount<STRATEGY>::kOut;
    constexpr int kWarps = CONSUMERS / 32;
    extern __shared__ unsigned char smem_raw[];
    using Smem = PipeSmem<CONSUMERS, VPT, STAGES, STRATEGY>;
    Smem& sm = *reinterpret_cast<Smem*>((reinterpret_cast<uintptr_t>(smem_raw) + 127) & ~static_cast<uintptr_t>(127));

    const bool is_producer = threadIdx.x >= CONSUMERS;
    if (threadIdx.x == 0) {
#pragma unroll
        for (int s = 0; s < STAGES; ++s) {
            pipe::mbar_init(&sm.full[s], 1);
            pipe::mbar_init(&sm.done[s], kWarps);
        }
        pipe::mbar_init(&sm.red_full, kWarps);
        pipe::mbar_init(&sm.red_free, 1);
        pipe::mbar_init_fence();
    }
    __syncthreads();

    double dot = 0.0, sq = 0.0;
    uint32_t lost = 0;
    const StepScalars& k = p.k;
    uint32_t it = 0;          // running tile number of this block; both roles count the same sequence
    bool alive = true;

    if (is_producer) {
        if (threadIdx.x == CONSUMERS) {
            // what sits in each stage, so that it can be stored out once the consumers are done with it
            uint16_t* held_out[STAGES][5];
            uint32_t held_bytes[STAGES];
            uint32_t held_tensor[STAGES];      // for the replica copies of theta (multi-tensor plans only)
            uint64_t held_elem[STAGES];
#pragma unroll
            for (int s = 0; s < STAGES; ++s) {
                held_bytes[s] = 0;
                held_tensor[s] = 0;
                held_elem[s] = 0;
            }
            // theta of a finished tile also goes to every replica registered with the plan
            auto store_replicas = [&](int s) {
                if constexpr (!FLAT) {
                    for (int r = 0; r < p.num_replicas; ++r)
                        pipe::bulk_store(replica_ptr(p, r, held_tensor[s], held_elem[s]), sm.data[s][0], held_bytes[s]);
                }
            };

            for (uint64_t c = blockIdx.x; c < p.num_chunks && alive; c += gridDim.x) {
                TensorRec t;
                uint64_t start;
                uint32_t tensor_id = 0;
                if (FLAT) {
                    t = p.flat;
                    start = c * p.chunk_elems;
                } else {
                    const ChunkRec cr = p.chunks[c];
                    tensor_id = cr.tensor;
                    t = p.tensors[cr.tensor];
                    start = static_cast<uint64_t>(cr.index) * p.chunk_elems;
                }
                const uint64_t left = t.n - start;
                const uint32_t len = left < p.chunk_elems ? static_cast<uint32_t>(left) : p.chunk_elems;
                for (uint32_t off = 0; off < len && alive; off += kTile, ++it) {
                    const int s = it % STAGES;
                    const uint32_t use = it / STAGES;
                    if (use > 0) {   // the stage still holds tile it - STAGES: wait for it, send it home
                        alive = pipe::mbar_wait(&sm.done[s], (use - 1) & 1u, 10u + s, &g_pipeline_fault);
                        if (!alive) break;
                        if (held_bytes[s]) {
#pragma unroll
                            for (int a = 0; a < NOUT; ++a) pipe::bulk_store(held_out[s][a], sm.data[s][a], held_bytes[s]);
                            store_replicas(s);
                            pipe::bulk_commit();
                            pipe::bulk_wait_read_all();   // the stage may be overwritten once it has been read out
                        }
                    }
                    const uint32_t tl = (len - off) < static_cast<uint32_t>(kTile) ? (len - off) : kTile;
                    const bool bulk = t.aligned && tl == static_cast<uint32_t>(kTile);
                    if (bulk) {
                        const uint16_t* g;
                        tile_pointers<STRATEGY>(t, start + off, held_out[s], g);
                        held_bytes[s] = kTile * 2;
                        held_elem[s] = start + off;
                        held_tensor[s] = tensor_id;
                        pipe::mbar_arrive_expect_tx(&sm.full[s], NIN * kTile * 2);
#pragma unroll
                        for (int a = 0; a < NOUT; ++a) pipe::bulk_load(sm.data[s][a], held_out[s][a], kTile * 2, &sm.full[s]);
                        pipe::bulk_load(sm.data[s][NOUT], g, kTile * 2, &sm.full[s]);
                    } else {
                        held_bytes[s] = 0;
                        pipe::mbar_arrive(&sm.full[s]);
                    }
                }
            }
            // drain: the last min(it, STAGES) tiles are still in their stages
            const uint32_t tail = it < static_cast<uint32_t>(STAGES) ? it : STAGES;
            for (uint32_t j = it - tail; j < it && alive; ++j) {
                const int s = j % STAGES;
                alive = pipe::mbar_wait(&sm.done[s], (j / STAGES) & 1u, 20u + s, &g_pipeline_fault);
                if (!alive) break;
                if (held_bytes[s]) {
#pragma unroll
                    for (int a = 0; a < NOUT; ++a) pipe::bulk_store(held_out[s][a], sm.data[s][a], held_bytes[s]);
                    store_replicas(s);
                    pipe::bulk_commit();
                }
            }
            if (!alive) {
                // a wait gave up: loads already issued still land in shared memory; let them finish
                for (int s = 0; s < STAGES; ++s) {
                    const uint32_t armed = (it > static_cast<uint32_t>(s)) ? (it - 1 - s) / STAGES : 0;
                    if (it > static_cast<uint32_t>(s)) pipe::mbar_wait(&sm.full[s], armed & 1u, 30u + s, &g_pipeline_fault);
                }
            }
            pipe::bulk_wait_all();
        }
    } else {
        const int lane = threadIdx.x & 31;
        uint32_t chunks_done = 0;
        for (uint64_t c = blockIdx.x; c < p.num_chunks && alive; c += gridDim.x) {
            TensorRec t;
            uint64_t start;
            uint32_t tensor_id = 0;
            if (FLAT) {
                t = p.flat;
                start = c * p.chunk_elems;
            } else {
                const ChunkRec cr = p.chunks[c];
                tensor_id = cr.tensor;
                t = p.tensors[cr.tensor];
                start = static_cast<uint64_t>(cr.index) * p.chunk_elems;
            }
            const uint64_t left = t.n - start;
            const uint32_t len = left < p.chunk_elems ? static_cast<uint32_t>(left) : p.chunk_elems;
            for (uint32_t off = 0; off < len; off += kTile, ++it) {
                const int s = it % STAGES;
                // a wait that gives up must take the whole warp with it (the lanes meet again in __syncwarp)
                alive = __all_sync(0xFFFFFFFFu, pipe::mbar_wait(&sm.full[s], (it / STAGES) & 1u, 40u + s, &g_pipeline_fault));
                if (!alive) break;
                const uint32_t tl = (len - off) < static_cast<uint32_t>(kTile) ? (len - off) : kTile;
                if (t.aligned && tl == static_cast<uint32_t>(kTile)) {
#pragma unroll
                    for (int j = 0; j < VPT; ++j) {
                        const int e = (j * CONSUMERS + threadIdx.x) * 8;
                        if constexpr (FAST && STRATEGY != 4) {
                            Vec v = tile_vector_load<STRATEGY, kTile>(&sm.data[s][0][e]);
                            if (compute_vec_fast<STRATEGY, EDQ, VARIANT>(v, k, dot, sq, lost) == 0u) {
                                tile_vector_store<STRATEGY, kTile>(&sm.data[s][0][e], v);
                            } else {
                                // rare: the tile still holds the inputs; repeat the vector out of line
                                const VecSums r = careful_vector_in_tile<STRATEGY, EDQ, VARIANT, kTile>(&sm.data[s][0][e], k);
                                if (EDQ) {
                                    dot += r.dot;
                                    sq += r.sq;
                                    lost += r.lost;
                                }
                            }
                        } else {
                            Vec v = tile_vector_load<STRATEGY, kTile>(&sm.data[s][0][e]);
                            compute_vec<STRATEGY, EDQ, VARIANT>(v, k, 8, dot, sq, lost);
                            tile_vector_store<STRATEGY, kTile>(&sm.data[s][0][e], v);
                        }
                    }
                    pipe::fence_async_smem();      // shared-memory writes must be visible to the bulk store
                } else {
                    // straight from global memory: vectors where the tensor allows, elements otherwise
                    const uint32_t nvec = tl >> 3;
                    const int rem = static_cast<int>(tl & 7u);
                    const uint64_t base = start + off;
                    for (uint32_t i = threadIdx.x; i < nvec; i += CONSUMERS) {
                        Vec v;
                        if (t.aligned) load_vec<STRATEGY>(v, t, base + 8ull * i);
                        else load_elems<STRATEGY>(v, t, base + 8ull * i, 8);
                        compute_vec<STRATEGY, EDQ, VARIANT>(v, k, 8, dot, sq, lost);
                        if (t.aligned) store_vec<STRATEGY>(v, t, base + 8ull * i);
                        else store_elems<STRATEGY>(v, t, base + 8ull * i, 8);
                        if (!FLAT)
                            for (int r = 0; r < p.num_replicas; ++r) {
                                uint16_t* dst = replica_ptr(p, r, tensor_id, base + 8ull * i);
                                if (t.aligned) st_stream(dst, v.th);
                                else st_elems(dst, v.th, 8);
                            }
                    }
                    if (rem && threadIdx.x == (nvec % CONSUMERS)) {
                        Vec v;
                        load_elems<STRATEGY>(v, t, base + 8ull * nvec, rem);
                        compute_vec<STRATEGY, EDQ, VARIANT>(v, k, rem, dot, sq, lost);
                        store_elems<STRATEGY>(v, t, base + 8ull * nvec, rem);
                        if (!FLAT)
                            for (int r = 0; r < p.num_replicas; ++r)
                                st_elems(replica_ptr(p, r, tensor_id, base + 8ull * nvec), v.th, rem);
                    }
                }
                __syncwarp();
                if (lane == 0) pipe::mbar_arrive(&sm.done[s]);
            }
            if (EDQ && PER_CHUNK && alive) {
                // One record per chunk, summed over the consumers in a fixed order.  The hand-over of the
                // per-warp sums goes through two mbarriers with bounded waits (never a bar.sync, which
                // could not time out): red_full = "all warps have written", red_free = "thread 0 has read".
                unsigned long long lost64 = lost;
#pragma unroll
                for (int o = 16; o > 0; o >>= 1) {
                    dot += __shfl_down_sync(0xFFFFFFFFu, dot, o);
                    sq += __shfl_down_sync(0xFFFFFFFFu, sq, o);
                    lost64 += __shfl_down_sync(0xFFFFFFFFu, lost64, o);
                }
                if (chunks_done > 0)
                    alive = __all_sync(0xFFFFFFFFu, pipe::mbar_wait(&sm.red_free, (chunks_done - 1) & 1u, 50u, &g_pipeline_fault));
                if (alive) {
                    if (lane == 0) {
                        sm.red_dot[threadIdx.x >> 5] = dot;
                        sm.red_sq[threadIdx.x >> 5] = sq;
                        sm.red_lost[threadIdx.x >> 5] = lost64;
                        pipe::mbar_arrive(&sm.red_full);
                    }
                    if (threadIdx.x == 0) {
                        if (pipe::mbar_wait(&sm.red_full, chunks_done & 1u, 51u, &g_pipeline_fault)) {
                            double d = 0.0, q = 0.0;
                            unsigned long long l = 0;
#pragma unroll
                            for (int w = 0; w < kWarps; ++w) {
                                d += sm.red_dot[w];
                                q += sm.red_sq[w];
                                l += sm.red_lost[w];
                            }
                            p.chunk_partials[c] = EdqPartial{d, q, l, 0ull};
                            pipe::mbar_arrive(&sm.red_free);
                        }
                    }
                    __syncwarp();
                }
                dot = 0.0;
                sq = 0.0;
                lost = 0;
                ++chunks_done;
            }
        }
    }

    if (EDQ && !PER_CHUNK) {
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
        edq_publish_and_finish(p.fin, sm.finish, d, q, l, &g_pipeline_fault);
    }
}

}  // namespace collage
