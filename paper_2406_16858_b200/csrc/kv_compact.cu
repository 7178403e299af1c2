// Step 5 of the hot path: compaction of the accepted path's K/V rows (paper Section 2.1: rejected
// draft tokens are dropped; Appendix A: the cache is pre-allocated and extended in place).
//
// A thread owns one 16-byte column segment of one (layer, K|V, sequence): it loads that segment of
// every accepted row first and stores afterwards, so the in-place move is safe although sources and
// destinations overlap (destination j never exceeds source acc_path[j]).
#include "common.cuh"

namespace eagle2 {

constexpr int kCompactThreads = 128;
constexpr int kCompactMaxDepth = 16;

__device__ __forceinline__ bool path_is_valid(const int32_t* path, int len, int D, int m) {
    if (len < 0 || len > D) return false;
    int prev = -1;
    for (int j = 0; j < len; ++j) {
        const int src = path[j];
        if (src < j || src >= m || src <= prev) return false;
        prev = src;
    }
    return true;
}

__global__ void __launch_bounds__(kCompactThreads)
kv_compact_kernel(void* const* __restrict__ k_layers, void* const* __restrict__ v_layers,
                  const int64_t* __restrict__ kv_off, const int32_t* __restrict__ kv_len,
                  const int32_t* __restrict__ acc_path, const int32_t* __restrict__ acc_len, int m,
                  int D, int segs, int seg_blocks) {
    chain_wait();
    chain_release();
    const int b = blockIdx.x / seg_blocks;
    const int seg = (blockIdx.x % seg_blocks) * kCompactThreads + threadIdx.x;
    const int layer = blockIdx.y >> 1, which = blockIdx.y & 1;
    const int len = acc_len[b];
    const int32_t* path = acc_path + (long long)b * D;
    if (seg >= segs || len == 0 || !path_is_valid(path, len, D, m)) return;
    uint4* base = reinterpret_cast<uint4*>(which ? v_layers[layer] : k_layers[layer]) +
                  (kv_off[b] + kv_len[b]) * (long long)segs + seg;
    uint4 held[kCompactMaxDepth];
#pragma unroll
    for (int j = 0; j < kCompactMaxDepth; ++j)
        if (j < len) held[j] = base[(long long)path[j] * segs];
#pragma unroll
    for (int j = 0; j < kCompactMaxDepth; ++j)
        if (j < len && path[j] != j) base[(long long)j * segs] = held[j];
}

// Runs after the move (same stream): every block of the move kernel has read the old lengths.
// A sequence with an invalid path was left alone by the move and is reported here.
__global__ void kv_len_advance_kernel(int32_t* __restrict__ kv_len, const int32_t* __restrict__ acc_path,
                                      const int32_t* __restrict__ acc_len, int B, int m, int D,
                                      int32_t* d_status) {
    // No early release of the dependents here: whatever kernel follows may read the lengths before it
    // waits for its predecessor (the attention kernel does), so it must not start before they are final.
    chain_wait();
    const int b = blockIdx.x * blockDim.x + threadIdx.x;
    if (b >= B) return;
    const int len = acc_len[b];
    if (path_is_valid(acc_path + (long long)b * D, len, D, m))
        kv_len[b] += len;
    else
        raise_status(d_status, EAGLE2_STATUS_BAD_TREE);
}

}  // namespace eagle2

using namespace eagle2;

extern "C" int eagle2_kv_compact(void* const* k_layers, void* const* v_layers, int n_layers,
                                 const int64_t* kv_off, int32_t* kv_len, const int32_t* acc_path,
                                 const int32_t* acc_len, int B, int m, int D, int Hkv, int d,
                                 int32_t* d_status, eagle2_stream_t stream) {
    if (!k_layers || !v_layers || !kv_off || !kv_len || !acc_path || !acc_len || !d_status)
        return EAGLE2_ERR_NULL;
    if (B < 0 || n_layers < 0 || n_layers > 32767 || m < 1 || m > EAGLE2_MAX_M || D < 1 ||
        D > kCompactMaxDepth || Hkv < 1 || d < 1)
        return EAGLE2_ERR_SHAPE;
    const long long row_bytes = (long long)Hkv * d * 2;
    if (row_bytes % 16) return EAGLE2_ERR_ALIGN;
    if (B == 0) return EAGLE2_OK;
    cudaStream_t st = reinterpret_cast<cudaStream_t>(stream);
    const int segs = (int)(row_bytes / 16);
    const int seg_blocks = (segs + kCompactThreads - 1) / kCompactThreads;
    if (n_layers > 0) {
        if ((long long)B * seg_blocks > 0x7fffffffLL) return EAGLE2_ERR_SHAPE;
        dim3 grid((unsigned)(B * seg_blocks), (unsigned)(n_layers * 2));
        if (launch_chained(kv_compact_kernel, grid, dim3(kCompactThreads), 0, st, 1, k_layers, v_layers, kv_off,
                           kv_len, acc_path, acc_len, m, D, segs, seg_blocks) != EAGLE2_OK)
            return EAGLE2_ERR_CUDA;
    }
    return launch_chained(kv_len_advance_kernel, dim3((B + 127) / 128), dim3(128), 0, st, 1, kv_len, acc_path, acc_len,
                          B, m, D, d_status);
}
