// Vocabulary-row scanning pieces shared by the expansion and acceptance kernels: a chunk of one
// fp32 logit row is held in registers (128-bit coalesced loads), reduced to (max, sum of
// exponentials) and to its k largest entries by warp-shuffle selection plus a block-level merge.
#pragma once

#include "common.cuh"

namespace eagle2 {

constexpr int kScanThreads = 256;
constexpr int kScanWarps = kScanThreads / kWarp;

// Element j (0 <= j < 4*VPT) of this thread within chunk `chunk` of a row.
template <int VPT, bool VEC>
__device__ __forceinline__ int scan_elem_index(int chunk, int j) {
    constexpr int CH = kScanThreads * 4 * VPT;
    if (VEC) return chunk * CH + ((j >> 2) * kScanThreads + (int)threadIdx.x) * 4 + (j & 3);
    return chunk * CH + j * kScanThreads + (int)threadIdx.x;
}

// Loads the thread's 4*VPT elements; positions beyond V read as -inf.
template <int VPT, bool VEC>
__device__ __forceinline__ void scan_load(const float* __restrict__ row, int V, int chunk,
                                          float (&x)[4 * VPT]) {
    if (VEC) {
#pragma unroll
        for (int i = 0; i < VPT; ++i) {
            const int e0 = scan_elem_index<VPT, true>(chunk, 4 * i);
            float4 v = make_float4(-INFINITY, -INFINITY, -INFINITY, -INFINITY);
            if (e0 < V) v = __ldcs(reinterpret_cast<const float4*>(row + e0));
            x[4 * i + 0] = v.x;
            x[4 * i + 1] = v.y;
            x[4 * i + 2] = v.z;
            x[4 * i + 3] = v.w;
        }
    } else {
#pragma unroll
        for (int j = 0; j < 4 * VPT; ++j) {
            const int e = scan_elem_index<VPT, false>(chunk, j);
            x[j] = e < V ? __ldcs(row + e) : -INFINITY;
        }
    }
}

__device__ __forceinline__ float block_max_f32(float v, float* s_red /*[kScanWarps]*/) {
    v = warp_max_f32(v);
    __syncthreads();
    if ((threadIdx.x & 31) == 0) s_red[threadIdx.x >> 5] = v;
    __syncthreads();
    float r = s_red[0];
#pragma unroll
    for (int w = 1; w < kScanWarps; ++w) r = fmaxf(r, s_red[w]);
    return r;
}

__device__ __forceinline__ double block_sum_f64(double v, double* s_red /*[kScanWarps]*/) {
    v = warp_sum_f64(v);
    __syncthreads();
    if ((threadIdx.x & 31) == 0) s_red[threadIdx.x >> 5] = v;
    __syncthreads();
    double r = 0.0;
#pragma unroll
    for (int w = 0; w < kScanWarps; ++w) r += s_red[w];
    return r;
}

// k rounds of "take the warp-wide maximum key and retire it".  Keys are unique (they embed the
// index) except for the invalid key 0, so exactly one lane retires an entry per round.
template <int NKEY>
__device__ __forceinline__ void warp_select(unsigned long long (&key)[NKEY], int k,
                                            unsigned long long* dst /* k entries */) {
    const int lane = threadIdx.x & 31;
    for (int r = 0; r < k; ++r) {
        unsigned long long best = 0;
#pragma unroll
        for (int j = 0; j < NKEY; ++j) best = key[j] > best ? key[j] : best;
        const unsigned long long top = warp_max_u64(best);
#pragma unroll
        for (int j = 0; j < NKEY; ++j) key[j] = (key[j] == top) ? 0ull : key[j];
        if (lane == 0) dst[r] = top;
    }
}

// Block-level top-k of the keys held in registers.  s_keys: kScanWarps*EAGLE2_MAX_K entries.
// The k winners (descending; 0 = none) are written to out[0..k) by warp 0.
template <int NKEY>
__device__ __forceinline__ void block_topk(unsigned long long (&key)[NKEY], int k,
                                           unsigned long long* s_keys, unsigned long long* out) {
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    warp_select<NKEY>(key, k, s_keys + warp * EAGLE2_MAX_K);
    __syncthreads();
    if (warp == 0) {
        unsigned long long mine[kScanWarps];
#pragma unroll
        for (int t = 0; t < kScanWarps; ++t) {
            const int e = lane + 32 * t;  // entry e = (warp e / k, rank e % k)
            mine[t] = e < kScanWarps * k ? s_keys[(e / k) * EAGLE2_MAX_K + (e % k)] : 0ull;
        }
        warp_select<kScanWarps>(mine, k, out);
    }
}

// Sorts one value per lane across the warp, descending (lane 0 ends with the largest); NaN never
// wins a comparison and so sinks.
__device__ __forceinline__ float warp_sort_desc_f32(float v) {
    const int lane = threadIdx.x & 31;
#pragma unroll
    for (int size = 2; size <= 32; size <<= 1) {
#pragma unroll
        for (int stride = size >> 1; stride > 0; stride >>= 1) {
            const float other = __shfl_xor_sync(0xffffffffu, v, stride);
            const bool desc = (lane & size) == 0, lower = (lane & stride) == 0;
            v = (lower == desc) ? fmaxf(v, other) : fminf(v, other);
        }
    }
    return v;
}

// The same for one 64-bit key per lane.
__device__ __forceinline__ unsigned long long warp_sort_desc_u64(unsigned long long v) {
    const int lane = threadIdx.x & 31;
#pragma unroll
    for (int size = 2; size <= 32; size <<= 1) {
#pragma unroll
        for (int stride = size >> 1; stride > 0; stride >>= 1) {
            const unsigned long long other = __shfl_xor_sync(0xffffffffu, v, stride);
            const bool desc = (lane & size) == 0, lower = (lane & stride) == 0;
            const unsigned long long hi = v > other ? v : other, lo = v > other ? other : v;
            v = (lower == desc) ? hi : lo;
        }
    }
    return v;
}

// Choose elements per chunk (as float4 per thread: 1, 2 or 4) so that a launch fills the GPU when
// it can and no row is cut into more pieces than the merge step can hold.
inline int scan_pick_vpt(long long rows, int V) {
    const long long want_blocks = 2LL * sm_count();
    for (int vpt = 4; vpt >= 2; vpt >>= 1) {
        const long long chunks = (V + kScanThreads * 4 * vpt - 1) / (kScanThreads * 4 * vpt);
        if (rows * chunks >= want_blocks) return vpt;
    }
    return 1;
}
inline int scan_chunks(int V, int vpt) {
    return (V + kScanThreads * 4 * vpt - 1) / (kScanThreads * 4 * vpt);
}

}  // namespace eagle2
