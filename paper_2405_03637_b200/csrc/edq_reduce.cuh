// End of a step kernel's EDQ reduction (Eq. 3) without a second launch.
//
// Every block publishes its partial sums, then draws a ticket from a counter in the caller's
// workspace.  Nobody waits for anybody: the block that draws the last ticket knows that all other
// partials are already in memory, adds them up in index order (so the result does not depend on
// which block happened to come last) and writes the collage_edq_t record.  atomicInc wraps the
// counter back to zero with the last ticket, so the workspace is ready for the next call; it has
// to be zero before the first one (collage_workspace_init).
#pragma once
#include "host_common.cuh"

namespace collage {

// What the last block needs to finish the reduction.  `out == nullptr` means: no EDQ in this launch.
struct EdqFinish {
    EdqPartial* partials;        // one slot per block (workspace)
    unsigned int* ticket;        // counter behind the partials (workspace), zero between launches
    collage_edq_t* out;          // the record
    unsigned long long n;        // parameters covered by this launch
    int accumulate;              // add to the record's current sums (a step issued in slabs)
};

constexpr int kFinishThreads = 256;

// Scratch in shared memory for the last block's sum.
struct EdqFinishSmem {
    double dot[kFinishThreads / 32], sq[kFinishThreads / 32];
    unsigned long long lost[kFinishThreads / 32];
    unsigned int is_last, fault;
};

// Called by EVERY thread of the block (it contains block-wide barriers) once the block's own sums
// (d, q, l: meaningful in thread 0 only) are complete.  blockDim.x >= kFinishThreads.
// `fault_word` is the device word in which bounded waits record that they gave up; its value goes
// into the record so that the caller sees a torn step without another synchronisation.
__device__ __forceinline__ void edq_publish_and_finish(const EdqFinish& f, EdqFinishSmem& sm, double d, double q,
                                                       unsigned long long l, const unsigned int* fault_word) {
    if (threadIdx.x == 0) {
        f.partials[blockIdx.x] = EdqPartial{d, q, l, 0ull};
        __threadfence();                                    // the partial is visible before the ticket is drawn
        const unsigned int last = gridDim.x - 1;
        unsigned int t = atomicInc(f.ticket, last);
        // A value above `last` was never a count: the word was not zeroed.  atomicInc has just reset
        // it, so drawing once more puts this block into a correct sequence.
        if (t > last) t = atomicInc(f.ticket, last);
        sm.is_last = (t == last) ? 1u : 0u;
    }
    __syncthreads();
    if (!sm.is_last) return;
    __threadfence();                                        // other blocks' partials, written before their tickets
    double sd = 0.0, sq = 0.0;
    unsigned long long sl = 0;
    // one thread fetches the fault word while the others fetch the partials (every block's waits are over)
    if (threadIdx.x == kFinishThreads - 1) sm.fault = fault_word ? *reinterpret_cast<const volatile unsigned int*>(fault_word) : 0u;
    if (threadIdx.x < kFinishThreads) {
        for (unsigned int i = threadIdx.x; i < gridDim.x; i += kFinishThreads) {    // index order per thread
            const double2 a = __ldcg(reinterpret_cast<const double2*>(&f.partials[i]));
            sd += a.x;
            sq += a.y;
            sl += __ldcg(&f.partials[i].lost);
        }
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) {
            sd += __shfl_down_sync(0xFFFFFFFFu, sd, o);
            sq += __shfl_down_sync(0xFFFFFFFFu, sq, o);
            sl += __shfl_down_sync(0xFFFFFFFFu, sl, o);
        }
        if ((threadIdx.x & 31) == 0) {
            sm.dot[threadIdx.x >> 5] = sd;
            sm.sq[threadIdx.x >> 5] = sq;
            sm.lost[threadIdx.x >> 5] = sl;
        }
    }
    __syncthreads();
    if (threadIdx.x == 0) {
        double dot = 0.0, sumsq = 0.0;
        unsigned long long lost = 0, n = f.n;
#pragma unroll
        for (int w = 0; w < kFinishThreads / 32; ++w) {
            dot += sm.dot[w];
            sumsq += sm.sq[w];
            lost += sm.lost[w];
        }
        unsigned long long fault = sm.fault;
        if (f.accumulate) {
            dot += f.out->dot;
            sumsq += f.out->sumsq;
            lost += f.out->lost;
            n += f.out->n;
            if (!fault) fault = f.out->fault;
        }
        f.out->dot = dot;
        f.out->sumsq = sumsq;
        f.out->edq = sumsq > 0.0 ? dot / sqrt(sumsq) : 0.0;
        f.out->n = n;
        f.out->lost = lost;
        f.out->fault = fault;
    }
}

}  // namespace collage
