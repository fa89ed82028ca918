// Host-side helpers shared by the library's entry points: device checks, overlap checks, the
// double -> bfloat16 rounding used for the step's scalars, and the EDQ partial-sum layout.
#pragma once
#include <algorithm>
#include <atomic>
#include <cmath>
#include <cstdint>
#include <cstring>
#include <utility>
#include <vector>
#include <cuda_runtime.h>

#include "../../include/collage.h"

namespace collage {

// One EDQ partial per thread block, summed by the finalize kernel in index order.
struct EdqPartial {
    double dot, sq;
    unsigned long long lost, pad;
};
constexpr int kMaxGrid = 4096;                       // upper bound on persistent grid size
// workspace layout: kMaxGrid partials, then the ticket counter of the last-block reduction
constexpr size_t kTicketOffset = sizeof(EdqPartial) * kMaxGrid;
constexpr size_t kWorkspaceBytes = kTicketOffset + 64;

struct DeviceInfo {
    int sm_count = 0;
    int cc_major = 0;
};

// Facts about the current device, looked up once per device.  Returns COLLAGE_ERR_ARCH unless
// the device is compute capability 10.x: the kernels are built for sm_100a only and there is
// no fallback.  Safe to call from several host threads at once: the cached word is written with
// one atomic store after the (idempotent) lookup, so racing first calls store the same value.
inline collage_status_t current_device(DeviceInfo* out) {
    static std::atomic<uint32_t> cache[64];            // 0 = unknown, else 1 | sm_count << 1 | cc_major << 17
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess) return COLLAGE_ERR_CUDA;
    if (dev < 0 || dev >= 64) return COLLAGE_ERR_CUDA;
    uint32_t w = cache[dev].load(std::memory_order_acquire);
    if (w == 0) {
        int sm = 0, major = 0;
        if (cudaDeviceGetAttribute(&sm, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess) return COLLAGE_ERR_CUDA;
        if (cudaDeviceGetAttribute(&major, cudaDevAttrComputeCapabilityMajor, dev) != cudaSuccess) return COLLAGE_ERR_CUDA;
        w = 1u | (static_cast<uint32_t>(sm & 0xFFFF) << 1) | (static_cast<uint32_t>(major & 0xFF) << 17);
        cache[dev].store(w, std::memory_order_release);
    }
    out->sm_count = static_cast<int>((w >> 1) & 0xFFFF);
    out->cc_major = static_cast<int>((w >> 17) & 0xFF);
    return out->cc_major == 10 ? COLLAGE_OK : COLLAGE_ERR_ARCH;
}

// Byte ranges [begin, end) of the arrays of one call; overlap of any two is an error.
struct ByteRange {
    uintptr_t begin, end;
};

inline void push_range(std::vector<ByteRange>& v, const void* p, uint64_t n_elems) {
    if (p && n_elems) v.push_back({reinterpret_cast<uintptr_t>(p), reinterpret_cast<uintptr_t>(p) + 2 * n_elems});
}

inline void push_bytes(std::vector<ByteRange>& v, const void* p, uint64_t bytes) {
    if (p && bytes) v.push_back({reinterpret_cast<uintptr_t>(p), reinterpret_cast<uintptr_t>(p) + bytes});
}

// Does [p, p + bytes) overlap any range of `sorted` (sorted by begin, pairwise disjoint)?
inline bool overlaps_sorted(const std::vector<ByteRange>& sorted, const void* p, uint64_t bytes) {
    if (!p || !bytes || sorted.empty()) return false;
    const uintptr_t b = reinterpret_cast<uintptr_t>(p), e = b + bytes;
    // first range that begins at or after e; the one before it is the only candidate that can reach past b
    auto it = std::lower_bound(sorted.begin(), sorted.end(), e, [](const ByteRange& r, uintptr_t x) { return r.begin < x; });
    return it != sorted.begin() && (it - 1)->end > b;
}

inline bool any_overlap(std::vector<ByteRange>& v) {
    std::sort(v.begin(), v.end(), [](const ByteRange& a, const ByteRange& b) { return a.begin < b.begin; });
    for (size_t i = 1; i < v.size(); ++i)
        if (v[i].begin < v[i - 1].end) return true;
    return false;
}

// Nearest bfloat16 (ties to even) of a double, by integer manipulation of the IEEE-754 binary64
// encoding: the 53-bit significand is shifted down to the 8 bits bfloat16 keeps at that
// magnitude (fewer below 2^-126, gradual underflow), with one round-half-even decision.
inline uint16_t double_to_bf16_rn(double x) {
    uint64_t u;
    std::memcpy(&u, &x, sizeof u);
    const uint16_t sign = static_cast<uint16_t>((u >> 63) << 15);
    const uint64_t field = (u >> 52) & 0x7FF;
    const uint64_t frac = u & ((1ull << 52) - 1);
    if (field == 0x7FF) return sign | (frac ? 0x7FC0 : 0x7F80);
    if (field == 0) return sign;                        // binary64 subnormals are far below 2^-134
    const int e = static_cast<int>(field) - 1023;
    const uint64_t sig = frac | (1ull << 52);           // value = sig * 2^(e-52)
    const int shift = 45 + (e < -126 ? -126 - e : 0);   // low bits that do not fit
    if (shift >= 54) return sign;                       // below half of the smallest subnormal
    uint64_t q = sig >> shift;
    const uint64_t rem = sig & ((1ull << shift) - 1);
    const uint64_t half = 1ull << (shift - 1);
    if (rem > half || (rem == half && (q & 1))) ++q;
    // normal: q in [128, 256], a carry to 256 moves into the exponent by plain addition
    uint32_t bits = e >= -126 ? (static_cast<uint32_t>(e + 127) << 7) + static_cast<uint32_t>(q - 128)
                              : static_cast<uint32_t>(q);
    if (bits >= 0x7F80) bits = 0x7F80;                  // overflow
    return sign | static_cast<uint16_t>(bits);
}

inline double bf16_to_double(uint16_t h) {
    const uint32_t w = static_cast<uint32_t>(h) << 16;
    float f;
    std::memcpy(&f, &w, sizeof f);
    return static_cast<double>(f);
}

inline bool hyper_in_range(const collage_hyper_t* h) {
    auto nonneg = [](double v) { return std::isfinite(v) && v >= 0.0; };
    auto unit = [](double v) { return std::isfinite(v) && v >= 0.0 && v < 1.0; };
    return nonneg(h->lr) && nonneg(h->eps) && nonneg(h->weight_decay) && unit(h->beta1) && unit(h->beta2);
}

}  // namespace collage
