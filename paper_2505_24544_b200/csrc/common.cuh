// Shared device helpers of the Beagle draft-head kernels (sm_100a).
#pragma once
#include <cuda_bf16.h>
#include <cuda_runtime.h>
#include <stdint.h>

namespace beagle {

constexpr int kMaxCallBatch = 64;   // rows of one serve-time call (matches BEAGLE_MAX_CALL_BATCH)

typedef __nv_bfloat16 bf16;

// Per-call batch description, passed BY VALUE in the kernel parameters so that no host->device
// copy and no device-side state is needed for the host's cache bookkeeping.
struct BatchMeta {
    int32_t slot[kMaxCallBatch];     // cache slot of batch row b
    int32_t kv_len[kMaxCallBatch];   // keys visible to row b (true + draft states in the cache)
};
struct RowMap {
    int32_t idx[kMaxCallBatch];
};

template <typename T> struct VecOf;                     // 16-byte vector of T
template <> struct VecOf<float> { static constexpr int N = 4; };
template <> struct VecOf<bf16>  { static constexpr int N = 8; };

__device__ __forceinline__ float bf16_bits_to_float(uint32_t hi16) { return __uint_as_float(hi16 << 16); }

// 16-byte read-only (non-coherent) load that does not allocate in L1.  ONLY for data that no kernel writes while the
// reading kernel may be resident: weights, logits handed in by the caller, cache rows of true states.
__device__ __forceinline__ uint4 ld_stream16(const void* p) {
    uint4 v;
    asm volatile("ld.global.nc.L1::no_allocate.v4.u32 {%0,%1,%2,%3}, [%4];"
                 : "=r"(v.x), "=r"(v.y), "=r"(v.z), "=r"(v.w) : "l"(p));
    return v;
}
// 16-byte read-only (non-coherent) cached load: same restriction as ld_stream16.
__device__ __forceinline__ uint4 ld_cached16(const void* p) { return __ldg(reinterpret_cast<const uint4*>(p)); }
// 16-byte ordinary (coherent) loads for everything a kernel of the same launch chain writes -- activations, Q, the slots'
// previous states, cache rows of the draft tail: with programmatic dependent launch the reader may already be resident
// while the producer still runs, which the non-coherent path does not allow.  To be issued after pdl_wait().
__device__ __forceinline__ uint4 ld_act16(const void* p) {
    uint4 v;
    asm volatile("ld.global.v4.u32 {%0,%1,%2,%3}, [%4];" : "=r"(v.x), "=r"(v.y), "=r"(v.z), "=r"(v.w) : "l"(p) : "memory");
    return v;
}
__device__ __forceinline__ uint32_t ld_act32(const void* p) {
    uint32_t v;
    asm volatile("ld.global.u32 %0, [%1];" : "=r"(v) : "l"(p) : "memory");
    return v;
}
__device__ __forceinline__ uint4 ld_act_stream16(const void* p) {       // the same, without allocating in L1 (read once)
    uint4 v;
    asm volatile("ld.global.L1::no_allocate.v4.u32 {%0,%1,%2,%3}, [%4];"
                 : "=r"(v.x), "=r"(v.y), "=r"(v.z), "=r"(v.w) : "l"(p) : "memory");
    return v;
}

template <typename T> __device__ __forceinline__ void unpack16(const uint4& v, float* f);
template <> __device__ __forceinline__ void unpack16<float>(const uint4& v, float* f) {
    f[0] = __uint_as_float(v.x); f[1] = __uint_as_float(v.y); f[2] = __uint_as_float(v.z); f[3] = __uint_as_float(v.w);
}
template <> __device__ __forceinline__ void unpack16<bf16>(const uint4& v, float* f) {
    f[0] = __uint_as_float(v.x << 16); f[1] = __uint_as_float(v.x & 0xffff0000u);
    f[2] = __uint_as_float(v.y << 16); f[3] = __uint_as_float(v.y & 0xffff0000u);
    f[4] = __uint_as_float(v.z << 16); f[5] = __uint_as_float(v.z & 0xffff0000u);
    f[6] = __uint_as_float(v.w << 16); f[7] = __uint_as_float(v.w & 0xffff0000u);
}

template <typename T> __device__ __forceinline__ float to_float(T v);
template <> __device__ __forceinline__ float to_float<float>(float v) { return v; }
template <> __device__ __forceinline__ float to_float<bf16>(bf16 v) { return __bfloat162float(v); }
template <typename T> __device__ __forceinline__ T from_float(float v);
template <> __device__ __forceinline__ float from_float<float>(float v) { return v; }
template <> __device__ __forceinline__ bf16 from_float<bf16>(float v) { return __float2bfloat16_rn(v); }

__device__ __forceinline__ float warp_sum(float v) {
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
    return v;
}
__device__ __forceinline__ float warp_max(float v) {
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) v = fmaxf(v, __shfl_xor_sync(0xffffffffu, v, o));
    return v;
}

// Arg-max key: larger key <=> larger value, ties resolved to the LOWER index.  NaN is mapped to
// -inf (never wins) and -0 to +0 (equal to +0, as a floating-point compare sees them).
__device__ __forceinline__ unsigned long long argmax_key(float v, int idx) {
    if (v != v) v = -INFINITY;
    v = v + 0.0f;
    uint32_t u = __float_as_uint(v);
    u = (u & 0x80000000u) ? ~u : (u | 0x80000000u);
    return (static_cast<unsigned long long>(u) << 32) | static_cast<unsigned long long>(0xffffffffu - static_cast<uint32_t>(idx));
}
__device__ __forceinline__ int argmax_key_index(unsigned long long key) {
    return static_cast<int>(0xffffffffu - static_cast<uint32_t>(key & 0xffffffffull));
}
__device__ __forceinline__ unsigned long long warp_max_u64(unsigned long long k) {
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) {
        unsigned long long other = __shfl_xor_sync(0xffffffffu, k, o);
        k = other > k ? other : k;
    }
    return k;
}

__device__ __forceinline__ float silu_f(float u) { return u / (1.0f + __expf(-u)); }

// Bounds-checking build (-DBEAGLE_BOUNDS_CHECK; a second library, built with relocatable device code, for tests).
// Every access whose index comes from the host's per-call metadata -- cache slot and position of a scatter or a chunk,
// row maps, token ids -- is guarded by BEAGLE_IN_BOUNDS(condition): a violation raises the device error word of the
// context that was set up last (value 2, reported by beagle_check_device) and the access is SKIPPED; nothing traps.
// In the ordinary build the macro is the constant `true` and no code is generated.
#ifdef BEAGLE_BOUNDS_CHECK
extern __device__ int* g_bounds_word;          // bound by the context's device set-up (api.cu)
extern __device__ int g_bounds_slots;          // max_slots of that context
__device__ __forceinline__ bool bounds_report(bool ok) {
    if (!ok && g_bounds_word != nullptr) atomicExch(g_bounds_word, 2);
    return ok;
}
#define BEAGLE_IN_BOUNDS(cond) (::beagle::bounds_report(cond))
#define BEAGLE_SLOT_OK(slot) ((slot) >= 0 && (slot) < ::beagle::g_bounds_slots)
#else
#define BEAGLE_IN_BOUNDS(cond) true
#define BEAGLE_SLOT_OK(slot) true
#endif

// Programmatic dependent launch.  The serve-time kernels are launched so that a kernel may start
// while its predecessor in the stream is still draining: everything before pdl_wait() must touch
// only memory that no kernel of the chain writes (weights, the stable part of the K/V cache) and
// must write no global memory; pdl_wait() returns once the predecessor has completed and its
// writes are visible.  Loads rule: the non-coherent loads (ld.global.nc, __ldg: ld_stream16 /
// ld_cached16) are for weights and true-state cache rows only; whatever a kernel of the chain
// writes (activations, Q, h_slot, draft-tail cache rows, split partials) is read with ordinary
// loads (ld_act16 / ld_act32 / ld_act_stream16, TMA, or plain C++ loads through pointers that are
// NOT declared `const ... __restrict__` -- that pair lets the compiler pick the non-coherent path
// by itself) issued after pdl_wait().  Every kernel launched this way calls pdl_wait() on every thread, so that a
// kernel's completion implies the completion of all kernels before it.  Both are no-ops for a
// plain launch.
__device__ __forceinline__ void pdl_launch_dependents() { asm volatile("griddepcontrol.launch_dependents;" ::: "memory"); }
__device__ __forceinline__ void pdl_wait() { asm volatile("griddepcontrol.wait;" ::: "memory"); }
__device__ __forceinline__ void prefetch_l2(const void* p) { asm volatile("prefetch.global.L2 [%0];" ::"l"(p)); }

// Function attributes are per device.  One of these per kernel instantiation (a function-local static) remembers on which
// devices the dynamic shared-memory limit has been raised, so a process that drives several GPUs sets it on each.
struct PerDeviceOnce {
    static constexpr int kMaxDevices = 64;
    bool done[kMaxDevices] = {};
    // True when `fn` has been applied on the current device (now or earlier); false when it failed.
    template <typename F>
    bool ensure(F fn) {
        int dev = 0;
        if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= kMaxDevices) return false;
        if (done[dev]) return true;
        if (!fn()) return false;
        done[dev] = true;
        return true;
    }
};

// Launch with the programmatic-stream-serialization attribute (falls back to a plain launch if the
// attribute is refused).
template <typename... KArgs, typename... Args>
inline void launch_pdl(void (*kernel)(KArgs...), dim3 grid, dim3 block, size_t smem, cudaStream_t stream, Args&&... args) {
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = grid;
    cfg.blockDim = block;
    cfg.dynamicSmemBytes = smem;
    cfg.stream = stream;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr;
    cfg.numAttrs = 1;
    if (cudaLaunchKernelEx(&cfg, kernel, static_cast<KArgs>(args)...) != cudaSuccess) {
        cudaGetLastError();
        cfg.numAttrs = 0;
        cudaLaunchKernelEx(&cfg, kernel, static_cast<KArgs>(args)...);
    }
}

}  // namespace beagle
