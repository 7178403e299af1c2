// Shared device/host helpers of the sm_100a library (no arithmetic of the method lives here).
#pragma once

#include <cuda_runtime.h>
#include <stdint.h>

#include "eagle2.h"

namespace eagle2 {

constexpr int kWarp = 32;
constexpr size_t kWsAlign = 256;

__host__ __device__ inline size_t round_up(size_t x, size_t a) { return (x + a - 1) / a * a; }
__host__ __device__ inline long long nodes_of(int k, int D) {
    return (long long)k + (long long)(D - 1) * k * k;
}

// Every operation's workspace layout starts with the same arrival-counter region, zeroed once by
// eagle2_workspace_init and left at zero by every kernel: one ticket per sequence.
__host__ __device__ inline size_t counters_bytes(int B) { return round_up(sizeof(int) * (size_t)B, kWsAlign); }

inline bool aligned(const void* p, size_t a) { return (reinterpret_cast<uintptr_t>(p) % a) == 0; }

inline int launch_result() { return cudaGetLastError() == cudaSuccess ? EAGLE2_OK : EAGLE2_ERR_CUDA; }

// Bound, in clock cycles, that the next launches give their device-side waits (eagle2_set_wait_limit).
long long wait_limit_cycles();

// Streaming multiprocessors of the current device, queried once per device ordinal and kept for
// the life of the process.  Launch plans and workspace sizes are both derived from it, so they
// agree.  Without a usable device (a size query on a machine that has none) the B200's 148.
inline int sm_count() {
    constexpr int kMaxDevices = 64, kDefault = 148;
    static int cached[kMaxDevices] = {};
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= kMaxDevices) {
        cudaGetLastError();
        return kDefault;
    }
    if (cached[dev] == 0) {
        int sms = 0;
        if (cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess || sms < 1) {
            cudaGetLastError();
            sms = kDefault;
        }
        cached[dev] = sms;
    }
    return cached[dev];
}

// Every kernel of the library is launched with programmatic stream serialisation and begins with
// chain_wait(): it may be scheduled while its predecessor in the stream is still draining, and it
// touches no global memory before that predecessor (and, by induction, everything before it) has
// completed.  chain_release() lets the successor be scheduled in turn.  After a kernel that never
// releases, the successor simply starts when that kernel ends.
#ifdef __CUDACC__
__device__ __forceinline__ void chain_wait() { asm volatile("griddepcontrol.wait;" ::: "memory"); }
__device__ __forceinline__ void chain_release() { asm volatile("griddepcontrol.launch_dependents;" ::: "memory"); }

template <typename... KArgs, typename... Args>
inline int launch_chained(void (*kernel)(KArgs...), dim3 grid, dim3 block, size_t smem, cudaStream_t stream,
                          unsigned cluster_x, Args&&... args) {
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = grid;
    cfg.blockDim = block;
    cfg.dynamicSmemBytes = smem;
    cfg.stream = stream;
    cudaLaunchAttribute attr[2];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    attr[1].id = cudaLaunchAttributeClusterDimension;
    attr[1].val.clusterDim.x = cluster_x;
    attr[1].val.clusterDim.y = 1;
    attr[1].val.clusterDim.z = 1;
    cfg.attrs = attr;
    cfg.numAttrs = cluster_x > 1 ? 2 : 1;
    if (cudaLaunchKernelEx(&cfg, kernel, static_cast<KArgs>(args)...) != cudaSuccess) {
        cudaGetLastError();
        return EAGLE2_ERR_CUDA;
    }
    return EAGLE2_OK;
}
#endif

#ifdef __CUDACC__

__device__ __forceinline__ void raise_status(int32_t* d_status, int bits) {
    if (bits) atomicOr(d_status, bits);
}

// Monotone map float -> uint32 (larger float, larger code).  -0 is folded onto +0 first so that
// equal values always get equal codes; NaN maps to 0, the lowest code.
__device__ __forceinline__ uint32_t order_code(float x) {
    if (x != x) return 0u;
    const uint32_t u = __float_as_uint(x + 0.0f);
    return (u & 0x80000000u) ? ~u : (u | 0x80000000u);
}
__device__ __forceinline__ float order_decode(uint32_t c) {
    const uint32_t u = (c & 0x80000000u) ? (c & 0x7fffffffu) : ~c;
    return __uint_as_float(u);
}
// 64-bit selection key: value code in the high word, complemented index in the low word, so the
// maximum key is the largest value and, among equal values, the lowest index.  Valid keys are > 0.
__device__ __forceinline__ unsigned long long make_key(float x, uint32_t idx) {
    return ((unsigned long long)order_code(x) << 32) | (unsigned long long)(0xffffffffu - idx);
}
__device__ __forceinline__ uint32_t key_index(unsigned long long key) {
    return 0xffffffffu - (uint32_t)(key & 0xffffffffu);
}
__device__ __forceinline__ float key_value(unsigned long long key) {
    return order_decode((uint32_t)(key >> 32));
}

__device__ __forceinline__ unsigned long long warp_max_u64(unsigned long long v) {
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) {
        const unsigned long long other = __shfl_xor_sync(0xffffffffu, v, o);
        v = other > v ? other : v;
    }
    return v;
}
__device__ __forceinline__ float warp_max_f32(float v) {
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) v = fmaxf(v, __shfl_xor_sync(0xffffffffu, v, o));
    return v;
}
__device__ __forceinline__ float warp_sum_f32(float v) {
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
    return v;
}
__device__ __forceinline__ double warp_sum_f64(double v) {
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
    return v;
}
__device__ __forceinline__ double warp_max_f64(double v) {
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) v = fmax(v, __shfl_xor_sync(0xffffffffu, v, o));
    return v;
}

// Arrival ticket: returns true in exactly one block, the last of `expected` to arrive, after every
// other block's earlier global writes are visible to it.  The counter is left at zero.
__device__ __forceinline__ bool last_block_arrives(int* counter, int expected, int* smem_flag) {
    __syncthreads();
    if (threadIdx.x == 0) {
        __threadfence();  // cumulative: covers the writes the barrier ordered before it
        const int t = atomicAdd(counter, 1);
        const int last = (t == expected - 1);
        if (last) *counter = 0;
        *smem_flag = last;
    }
    __syncthreads();
    const bool last = *smem_flag != 0;
    if (last) __threadfence();
    return last;
}

#endif  // __CUDACC__

}  // namespace eagle2
