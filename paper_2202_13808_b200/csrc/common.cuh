// Shared device/host helpers of the DropIT CUDA library (sm_100a).
#pragma once

#include <cuda_runtime.h>
#include <stdint.h>

#include <atomic>

#include "dropit.h"

namespace dropit {

constexpr uint32_t kFullMask = 0xFFFFFFFFu;

// Per-dtype element traits.  An element's ordering key is its raw bits with the
// sign bit cleared (Sec. 3.3: selection is on absolute magnitude).
struct Bf16Traits {
    using elem_t = uint16_t;
    static constexpr int kElemBytes = 2;
    static constexpr int kVecElems = 8;      // elements per 16-byte vector
    static constexpr int kKeyBits = 15;
};
struct F32Traits {
    using elem_t = uint32_t;
    static constexpr int kElemBytes = 4;
    static constexpr int kVecElems = 4;
    static constexpr int kKeyBits = 31;
};

// Selection state shared by the histogram / threshold / compaction kernels.
// Lives at offset 0 of the compress workspace; zeroed at the start of a call.
struct SelectState {
    unsigned long long k_rem;      // retained count still to place inside the bucket chosen so far
    unsigned long long n_gt;       // #{key > T}
    unsigned long long quota;      // q = k - n_gt: ties at T that are retained (lowest flat indices)
    uint32_t prefix;               // high key digits decided so far
    uint32_t threshold;            // T
    uint32_t blocks_done[4];       // arrival counters, one per histogram pass
    uint32_t ticket;               // tile ticket of the compaction pass
    uint32_t reserved[19];
};
static_assert(sizeof(SelectState) == 128, "SelectState layout");

constexpr size_t kStateBytes = 256;           // SelectState, padded
constexpr int kHistThreads = 1024;
constexpr int kCompactThreads = 256;
constexpr int kCompactVecsPerThread = 4;
constexpr int kTileVecs = kCompactThreads * kCompactVecsPerThread;   // 1024 16-byte vectors per tile
constexpr int kSpinLimit = 1 << 20;           // bounded look-back wait

// Streaming 16-byte load that does not pollute L1.
__device__ __forceinline__ uint4 ld_stream(const uint4* p) {
    uint4 v;
    asm volatile("ld.global.nc.L1::no_allocate.v4.u32 {%0,%1,%2,%3}, [%4];"
                 : "=r"(v.x), "=r"(v.y), "=r"(v.z), "=r"(v.w)
                 : "l"(p));
    return v;
}

__device__ __forceinline__ unsigned long long ld_relaxed_u64(const unsigned long long* p) {
    unsigned long long v;
    asm volatile("ld.relaxed.gpu.global.u64 %0, [%1];" : "=l"(v) : "l"(p) : "memory");
    return v;
}

__device__ __forceinline__ void st_relaxed_u64(unsigned long long* p, unsigned long long v) {
    asm volatile("st.relaxed.gpu.global.u64 [%0], %1;" ::"l"(p), "l"(v) : "memory");
}

__device__ __forceinline__ uint32_t lane_id() { return threadIdx.x & 31; }

inline bool is_aligned16(const void* p) { return (reinterpret_cast<uintptr_t>(p) & 15u) == 0; }

inline size_t align_up(size_t v, size_t a) { return (v + a - 1) / a * a; }

// Number of SMs of the current device (cached per device id).
int sm_count();

// Index of the current device, or -1.
inline int current_device() {
    int dev = 0;
    return (cudaGetDevice(&dev) == cudaSuccess && dev >= 0) ? dev : -1;
}

// Kernel attributes (dynamic shared memory size, ...) belong to a device, not to the process: a call
// site keeps one of these and sets its attributes the first time it runs on each device.
struct PerDeviceOnce {
    std::atomic<bool> done[64];
    bool needed() const {
        const int dev = current_device();
        return dev < 0 || dev >= 64 || !done[dev].load(std::memory_order_acquire);
    }
    void mark() {
        const int dev = current_device();
        if (dev >= 0 && dev < 64) done[dev].store(true, std::memory_order_release);
    }
};

// A number that no earlier call of this process has used (and that another process is unlikely to
// have left in recycled memory): device-side barriers and ready flags that live in scratch memory
// nobody cleared tell this call's marks from stale ones by it.
uint32_t next_epoch();

// Polls that a bounded device-side wait makes before it gives up.  The defaults are far above any real
// wait; the environment variable DROPIT_TEST_SPIN_LIMIT (read at every call, tests only) overrides them
// so that the give-up paths can be exercised without hanging anything.
uint32_t spin_limit(uint32_t default_limit);

// Host-side shape of the compress workspace.
struct CompressPlan {
    int64_t n;
    int64_t k;
    int64_t n_tiles;
    size_t hist_offset, hist_bytes;
    size_t desc_offset, desc_bytes;
    size_t total_bytes;
};
CompressPlan make_compress_plan(int64_t n, int64_t k, dropit_dtype dtype);

inline cudaStream_t as_stream(void* s) { return reinterpret_cast<cudaStream_t>(s); }

// Kernel launches enqueued by this library since it was loaded (diagnostic counter).
extern std::atomic<unsigned long long> g_launch_count;

// Call once after every kernel launch.
inline dropit_status check_launch() {
    g_launch_count.fetch_add(1, std::memory_order_relaxed);
    return cudaGetLastError() == cudaSuccess ? DROPIT_OK : DROPIT_ERR_CUDA;
}

}  // namespace dropit
