// Library-level entry points: version, error strings, workspace sizing and initialisation.
#include <atomic>

#include "common.cuh"

namespace eagle2 {
static std::atomic<long long> g_wait_limit{0};  // 0: the built-in default
long long wait_limit_cycles() {
    const long long v = g_wait_limit.load(std::memory_order_relaxed);
    return v > 0 ? v : (1LL << 31);
}

size_t expand_workspace_bytes(int B, int V, int k);
size_t accept_workspace_bytes(int B, int V, int k, int D, int m);
size_t attention_workspace_bytes(int B, int m, int Hq, int Hkv, int d, int max_kv_len);
size_t lm_head_expand_workspace_bytes(int B, int V, int k);
}  // namespace eagle2

extern "C" int eagle2_version(void) { return 100; }

extern "C" const char* eagle2_strerror(int code) {
    switch (code) {
        case EAGLE2_OK: return "ok";
        case EAGLE2_ERR_NULL: return "a required pointer is NULL";
        case EAGLE2_ERR_SHAPE: return "a size is outside the supported range";
        case EAGLE2_ERR_ALIGN: return "a pointer or stride is not aligned as required";
        case EAGLE2_ERR_WORKSPACE: return "workspace missing, misaligned or too small";
        case EAGLE2_ERR_CUDA: return "the CUDA runtime refused the launch";
        case EAGLE2_ERR_STATIC_LIMIT: return "sizes need more scratch than the library's built-in buffer holds";
        default: return "unknown error code";
    }
}

extern "C" size_t eagle2_workspace_bytes(int op, int B, int V, int k, int D, int m, int Hq, int Hkv, int d,
                                         int max_kv_len) {
    if (B < 1) return 0;
    switch (op) {
        case EAGLE2_OP_EXPAND:
            if (V < 1 || k < 1 || k > EAGLE2_MAX_K) return 0;
            return eagle2::expand_workspace_bytes(B, V, k);
        case EAGLE2_OP_ACCEPT:
            if (V < 1 || k < 1 || D < 1 || m < 1) return 0;
            return eagle2::accept_workspace_bytes(B, V, k, D, m);
        case EAGLE2_OP_TREE_ATTENTION:
            if (m < 1 || Hq < 1 || Hkv < 1 || Hq % Hkv || (d != 64 && d != 128) || max_kv_len < 0) return 0;
            return eagle2::attention_workspace_bytes(B, m, Hq, Hkv, d, max_kv_len);
        case EAGLE2_OP_LM_HEAD_EXPAND:
            if (V < 1 || k < 1 || k > 16) return 0;
            return eagle2::lm_head_expand_workspace_bytes(B, V, k);
        default:
            return 0;  // rerank, tree mask and KV compaction work in place
    }
}

extern "C" long long eagle2_set_wait_limit(long long cycles) {
    const long long before = eagle2::wait_limit_cycles();
    eagle2::g_wait_limit.store(cycles > 0 ? cycles : 0, std::memory_order_relaxed);
    return before;
}

extern "C" int eagle2_workspace_init(void* ws, size_t ws_bytes, eagle2_stream_t stream) {
    if (ws_bytes == 0) return EAGLE2_OK;
    if (!ws) return EAGLE2_ERR_NULL;
    if (!eagle2::aligned(ws, eagle2::kWsAlign)) return EAGLE2_ERR_WORKSPACE;
    return cudaMemsetAsync(ws, 0, ws_bytes, reinterpret_cast<cudaStream_t>(stream)) == cudaSuccess
               ? EAGLE2_OK
               : EAGLE2_ERR_CUDA;
}
