// collage_edq_static: the EDQ reduction for callers that must not allocate.
//
// Same result as collage_edq, but the scratch memory for the per-block partial sums is not
// passed in: it lives in a file-scope device array of fixed size that every GPU loading this
// library carries until the process exits.  Nothing in this file calls cudaMalloc, cudaFree or
// any routine that allocates.
#include "host_common.cuh"
#include "mcf_device.cuh"

namespace collage {

void launch_edq_finalize(const EdqPartial* partials, int count, uint64_t n, collage_edq_t* out, cudaStream_t stream,
                         bool accumulate);

constexpr int kStaticThreads = 256;
constexpr int kStaticPartials = 2048;                        // 2048 x 32 B = 64 KiB of scratch
constexpr uint64_t kStaticMaxN = 1ull << 32;                 // elements; one block then reduces 2^21 of them
constexpr uint64_t kMinSegment = 2048;                       // elements reduced by one block, at least

// Elements per block for a tensor of n elements: enough blocks to fill the GPU at every size, never
// more than the scratch has slots, a whole number of 8-element vectors.  A function of n alone, so
// the grouping of the sums, and with it the result, is the same on every device.
inline uint64_t static_segment(uint64_t n) {
    uint64_t seg = (n + kStaticPartials - 1) / kStaticPartials;
    seg = (seg + 7) & ~7ull;
    return seg < kMinSegment ? kMinSegment : seg;
}

// The scratch itself.  In host code this name is only a handle for cudaGetSymbolAddress; it is
// not a device address and must never be passed to a kernel as one.
static __device__ __align__(256) EdqPartial g_static_partials[kStaticPartials];

struct StaticEdqArgs {
    const uint16_t* old_hi;
    const uint16_t* old_lo;
    const uint16_t* new_hi;
    const uint16_t* new_lo;
    const uint16_t* delta;
    uint64_t n;
    uint64_t segment;         // elements per block
    int aligned;
    EdqPartial* partials;     // device address of g_static_partials, looked up by the host
};

// Block b reduces elements [b * segment, (b+1) * segment) and overwrites partial b: every slot
// that the finalize kernel will read is written by this launch, so stale contents never matter.
template <bool HAS_LO>
__global__ void __launch_bounds__(kStaticThreads) edq_static_kernel(const __grid_constant__ StaticEdqArgs p) {
    const uint64_t seg_begin = blockIdx.x * p.segment;
    const uint64_t seg_end = (p.n - seg_begin < p.segment) ? p.n : seg_begin + p.segment;
    const uint64_t nvec = (seg_end - seg_begin + 7) >> 3;
    double dot = 0.0, sq = 0.0;
    unsigned long long lost = 0;
    for (uint64_t i = threadIdx.x; i < nvec; i += kStaticThreads) {
        const uint64_t off = seg_begin + i * 8;
        const uint64_t left = seg_end - off;
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
    __shared__ double s_dot[kStaticThreads / 32], s_sq[kStaticThreads / 32];
    __shared__ unsigned long long s_lost[kStaticThreads / 32];
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
        for (int x = 0; x < kStaticThreads / 32; ++x) {
            d += s_dot[x];
            q += s_sq[x];
            l += s_lost[x];
        }
        p.partials[blockIdx.x] = EdqPartial{d, q, l, 0ull};
    }
}

// Device address of the static scratch on the current device, looked up once per device.  Host
// threads racing on the first call look the same address up twice and store it twice.
static cudaError_t static_scratch(EdqPartial** out) {
    static std::atomic<EdqPartial*> address[64];
    int dev = 0;
    cudaError_t e = cudaGetDevice(&dev);
    if (e != cudaSuccess) return e;
    if (dev < 0 || dev >= 64) return cudaErrorInvalidDevice;
    EdqPartial* ptr = address[dev].load(std::memory_order_acquire);
    if (!ptr) {
        e = cudaGetSymbolAddress(reinterpret_cast<void**>(&ptr), g_static_partials);   // `dev` is current
        if (e != cudaSuccess) return e;
        address[dev].store(ptr, std::memory_order_release);
    }
    *out = ptr;
    return cudaSuccess;
}

}  // namespace collage

using namespace collage;

extern "C" collage_status_t collage_edq_static(const void* old_hi, const void* old_lo, const void* new_hi,
                                               const void* new_lo, const void* delta, uint64_t n,
                                               collage_edq_t* out_dev, void* stream) {
    if (!old_hi || !new_hi || !delta || !out_dev) return COLLAGE_ERR_NULL;
    if ((old_lo == nullptr) != (new_lo == nullptr)) return COLLAGE_ERR_NULL;
    if (n > kStaticMaxN) return COLLAGE_ERR_LIMIT;
    DeviceInfo dev;
    const collage_status_t st = current_device(&dev);
    if (st != COLLAGE_OK) return st;
    StaticEdqArgs p{};
    if (static_scratch(&p.partials) != cudaSuccess) return COLLAGE_ERR_CUDA;
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
    cudaStream_t cs = static_cast<cudaStream_t>(stream);
    p.segment = static_segment(n);
    const unsigned grid = static_cast<unsigned>((n + p.segment - 1) / p.segment);
    if (grid > 0) {
        if (old_lo) edq_static_kernel<true><<<grid, kStaticThreads, 0, cs>>>(p);
        else edq_static_kernel<false><<<grid, kStaticThreads, 0, cs>>>(p);
        if (cudaGetLastError() != cudaSuccess) return COLLAGE_ERR_CUDA;
    }
    launch_edq_finalize(p.partials, static_cast<int>(grid), n, out_dev, cs, false);
    return cudaGetLastError() == cudaSuccess ? COLLAGE_OK : COLLAGE_ERR_CUDA;
}
