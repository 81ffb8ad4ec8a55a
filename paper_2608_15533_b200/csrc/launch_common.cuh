// Host-side pieces shared by the translation units of the library: launch helpers, device facts, the
// expansion of a descriptor into template arguments, and the per-entry-point dispatch functions (each
// defined in a translation unit of its own so that the kernels compile in parallel).
#pragma once

#include <atomic>
#include <cstdint>
#include <cstdlib>
#include <map>
#include <tuple>
#include <mutex>
#include <type_traits>
#include <utility>

#include "common.cuh"
#include "validate.h"

namespace deltalog {

extern std::atomic<uint64_t> g_launches;  // kernels launched by the library in this process

inline int env_int(const char *name, int dflt) {
    const char *v = std::getenv(name);
    return v ? std::atoi(v) : dflt;
}
#if DELTALOG_TEST_HOOKS
inline int env_int_now(const char *name, int dflt) { return env_int(name, dflt); }  // read at every launch
#endif

inline int finish_launch() {
    g_launches.fetch_add(1, std::memory_order_relaxed);
    return cudaGetLastError() == cudaSuccess ? DELTALOG_OK : DELTALOG_ERR_CUDA;
}

// Raise the dynamic shared-memory limit of a kernel when a launch needs more than 48 KiB.  The limit
// only ever grows (per device), and it is raised to what launches have asked for, not to the device
// maximum: a kernel with static shared memory cannot be granted the whole opt-in size as dynamic.
template <typename K>
int ensure_smem(K kernel, size_t bytes) {
    if (bytes <= 48 * 1024) return DELTALOG_OK;
    static std::mutex mu;
    static std::map<std::pair<int, const void *>, size_t> granted;  // (device, kernel) -> bytes granted
    int dev = 0;
    cudaGetDevice(&dev);
    const auto key = std::make_pair(dev, reinterpret_cast<const void *>(kernel));
    std::lock_guard<std::mutex> lock(mu);
    size_t &g = granted[key];
    if (bytes <= g) return DELTALOG_OK;
    if (cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)bytes) != cudaSuccess) {
        cudaGetLastError();  // not sticky: leave the runtime clean for the caller
        return DELTALOG_ERR_CUDA;
    }
    g = bytes;
    return DELTALOG_OK;
}

// CTAs of a kernel that an SM holds at once with the given shared memory (after ensure_smem), looked up once per
// (device, kernel, size): the resident kernels size their grids by it.
template <typename K>
int resident_ctas(K kernel, int threads, size_t smem) {
    static std::mutex mu;
    static std::map<std::tuple<int, const void *, size_t>, int> known;
    int dev = 0;
    cudaGetDevice(&dev);
    const auto key = std::make_tuple(dev, reinterpret_cast<const void *>(kernel), smem);
    std::lock_guard<std::mutex> lock(mu);
    auto it = known.find(key);
    if (it != known.end()) return it->second;
    // Several CTAs of ~100 KB each only fit when the SM's L1 / shared-memory split is at its largest; left to itself the
    // driver may pick a split that holds one.
    if (cudaFuncSetAttribute(kernel, cudaFuncAttributePreferredSharedMemoryCarveout, cudaSharedmemCarveoutMaxShared) != cudaSuccess)
        cudaGetLastError();
    int n = 0;
    if (cudaOccupancyMaxActiveBlocksPerMultiprocessor(&n, kernel, threads, smem) != cudaSuccess) {
        cudaGetLastError();
        n = 0;
    }
    known[key] = n;
    return n;
}

// Launch with programmatic stream serialisation: the caller promised (DELTALOG_HINT_BASE_UNTOUCHED) that
// the kernel in front of this one on the stream does not write this state's base tiles, so this
// kernel's CTAs may start, and request base tiles, while that kernel is still retiring.
template <typename K, typename... Args>
int launch_chained(K kernel, int grid, int threads, size_t smem, cudaStream_t stream, Args... args) {
    cudaLaunchConfig_t lc = {};
    lc.gridDim = dim3(grid);
    lc.blockDim = dim3(threads);
    lc.dynamicSmemBytes = smem;
    lc.stream = stream;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    lc.attrs = attr;
    lc.numAttrs = 1;
    if (cudaLaunchKernelEx(&lc, kernel, args...) != cudaSuccess) {
        cudaGetLastError();
        return DELTALOG_ERR_CUDA;
    }
    g_launches.fetch_add(1, std::memory_order_relaxed);
    return DELTALOG_OK;
}

// Device facts needed to size the persistent kernel, queried once per device.
struct DeviceInfo {
    int sms = 0;
    int smem_per_sm = 0;
    int smem_optin = 0;
};
inline const DeviceInfo &device_info() {
    static DeviceInfo info[64];
    int dev = 0;
    cudaGetDevice(&dev);
    DeviceInfo &d = info[dev & 63];
    if (d.sms == 0) {
        cudaDeviceGetAttribute(&d.smem_per_sm, cudaDevAttrMaxSharedMemoryPerMultiprocessor, dev);
        cudaDeviceGetAttribute(&d.smem_optin, cudaDevAttrMaxSharedMemoryPerBlockOptin, dev);
        cudaDeviceGetAttribute(&d.sms, cudaDevAttrMultiProcessorCount, dev);
    }
    return d;
}


// Expand (op, d_k, d_v, io dtype) into the template instantiation: CALL(OP, DK, DV, IO).
#define DELTALOG_DISPATCH(desc, CALL)                                                        \
    do {                                                                                     \
        const int op_ = (desc)->op, dk_ = (desc)->d_k, dv_ = (desc)->d_v, io_ = (desc)->io_dtype; \
        if (op_ == DELTALOG_GDN) {                                                           \
            DELTALOG_DISPATCH_D(DELTALOG_GDN, dk_, dv_, io_, CALL);                          \
        } else if (op_ == DELTALOG_KDA) {                                                    \
            DELTALOG_DISPATCH_D(DELTALOG_KDA, dk_, dv_, io_, CALL);                          \
        } else if (op_ == DELTALOG_RETNET || op_ == DELTALOG_LINATTN) {                      \
            DELTALOG_DISPATCH_D(DELTALOG_RETNET, dk_, dv_, io_, CALL); /* linear attention: null gate */ \
        } else if (op_ == DELTALOG_GLA) {                                                    \
            DELTALOG_DISPATCH_D(DELTALOG_GLA, dk_, dv_, io_, CALL);                          \
        } else {                                                                             \
            DELTALOG_DISPATCH_D(DELTALOG_RWKV6, dk_, dv_, io_, CALL);                        \
        }                                                                                    \
    } while (0)
// (A translation unit may restrict itself to the 128 x 128 tiles, or to everything else, by defining
// DELTALOG_SHAPES_ONLY_128 / DELTALOG_SHAPES_NOT_128 before including this header.)
#if defined(DELTALOG_SHAPES_ONLY_128)
#define DELTALOG_DISPATCH_D(OP, dk_, dv_, io_, CALL)                                         \
    if (dk_ == 128 && dv_ == 128) {                                                          \
        DELTALOG_DISPATCH_IO(OP, 128, 128, io_, CALL);                                       \
    }
#elif defined(DELTALOG_SHAPES_NOT_128)
#define DELTALOG_DISPATCH_D(OP, dk_, dv_, io_, CALL)                                         \
    if (dk_ == 64 && dv_ == 64) {                                                            \
        DELTALOG_DISPATCH_IO(OP, 64, 64, io_, CALL);                                         \
    } else if (dk_ == 128 && dv_ == 64) {                                                    \
        DELTALOG_DISPATCH_IO(OP, 128, 64, io_, CALL);                                        \
    } else if (dk_ == 64 && dv_ == 128) {                                                    \
        DELTALOG_DISPATCH_IO(OP, 64, 128, io_, CALL);                                        \
    }
#else
#define DELTALOG_DISPATCH_D(OP, dk_, dv_, io_, CALL)                                         \
    if (dk_ == 64 && dv_ == 64) {                                                            \
        DELTALOG_DISPATCH_IO(OP, 64, 64, io_, CALL);                                         \
    } else if (dk_ == 128 && dv_ == 128) {                                                   \
        DELTALOG_DISPATCH_IO(OP, 128, 128, io_, CALL);                                       \
    } else if (dk_ == 128) {                                                                 \
        DELTALOG_DISPATCH_IO(OP, 128, 64, io_, CALL);                                        \
    } else {                                                                                 \
        DELTALOG_DISPATCH_IO(OP, 64, 128, io_, CALL);                                        \
    }
#endif
#define DELTALOG_DISPATCH_IO(OP, DK, DV, io_, CALL)                                          \
    if (io_ == DELTALOG_F32) { CALL(OP, DK, DV, float); } else { CALL(OP, DK, DV, __nv_bfloat16); }

// The value-side log keeps the I/O dtype where b = v (lossless).  For the delta rule it is fp32 by
// default; a 16-bit U log (descriptor ulog_dtype == io_dtype == BF16) is the reduced-precision variant.
// The dense base is fp32 unless the descriptor asks for the 16-bit state (16-bit I/O only).
#define DELTALOG_WITH_UL(OP, IO, desc, FN, DK, DV, ...)                                                    \
    do {                                                                                                  \
        if constexpr (!std::is_same<IO, float>::value) {                                                  \
            if ((desc)->base_dtype == DELTALOG_BF16) {                                                    \
                DELTALOG_WITH_UL_BT(OP, IO, __nv_bfloat16, desc, FN, DK, DV, __VA_ARGS__);                \
            }                                                                                             \
        }                                                                                                 \
        DELTALOG_WITH_UL_BT(OP, IO, float, desc, FN, DK, DV, __VA_ARGS__);                                 \
    } while (0)
#define DELTALOG_WITH_UL_BT(OP, IO, BT, desc, FN, DK, DV, ...)                                             \
    do {                                                                                                  \
        if constexpr (OpTraits<OP>::kDeltaRule) {                                                         \
            if constexpr (!std::is_same<IO, float>::value) {                                              \
                if ((desc)->ulog_dtype != DELTALOG_F32) return FN<OP, DK, DV, IO, IO, BT>(__VA_ARGS__);    \
            }                                                                                             \
            return FN<OP, DK, DV, IO, float, BT>(__VA_ARGS__);                                            \
        } else {                                                                                          \
            return FN<OP, DK, DV, IO, IO, BT>(__VA_ARGS__);                                               \
        }                                                                                                 \
    } while (0)

// One dispatch function per entry point: descriptor -> kernel instantiation -> launch.
int dispatch_decode_128(const deltalog_desc *desc, const StateArgs &st, const TokenArgs &tk, cudaStream_t s);    // 128 x 128 tiles
int dispatch_decode_other(const deltalog_desc *desc, const StateArgs &st, const TokenArgs &tk, cudaStream_t s);  // every other shape
int dispatch_decode_multi(const deltalog_desc *desc, const StateArgs &st, const TokenArgs &tk, int32_t T, cudaStream_t s);
int dispatch_fused_step(const deltalog_desc *desc, const StateArgs &st, const TokenArgs &tk, cudaStream_t s);
int dispatch_merge(const deltalog_desc *desc, const StateArgs &st, const int32_t *slot_idx, int32_t n, int32_t only_if_full,
                   cudaStream_t s);
int dispatch_reset_slots(const deltalog_desc *desc, const StateArgs &st, const int32_t *slot_idx, int32_t n, const float *S_init,
                         cudaStream_t s);
int dispatch_eager(const deltalog_desc *desc, void *S, int32_t *status, const TokenArgs &tk, cudaStream_t s);

}  // namespace deltalog
