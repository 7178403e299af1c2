// Step 2 of the hot path (paper Section 4.2): reranking of all candidate nodes by value, flattening
// of the selected subtree, and the ancestor attention mask with position ids.  The data is a few
// kilobytes per sequence, so each sequence is one thread block working in shared memory.
#include <math.h>

#include "common.cuh"

namespace eagle2 {

constexpr int kRerankThreads = 512;

// Monotone map double -> uint64 (larger value, larger code; -0 folded onto +0).  The caller has
// already replaced NaN.
__device__ __forceinline__ unsigned long long value_code(double x) {
    const unsigned long long u = (unsigned long long)__double_as_longlong(x + 0.0);
    return (u >> 63) ? ~u : (u | 0x8000000000000000ull);
}

// Row i of the ancestor mask (bit i and the bits of all ancestors of flat node i; a padding row has
// only its own bit) and its position id, from the selection's parent links in shared memory.
// Returns status bits.
__device__ __forceinline__ int mask_row(const int32_t* s_par, int i, int ns, int m, int b, int pos,
                                        uint64_t* __restrict__ mask_bits, uint8_t* __restrict__ mask_dense,
                                        int32_t* __restrict__ pos_ids) {
    const int W = (m + 63) / 64;
    uint64_t row[(EAGLE2_MAX_M + 63) / 64] = {0, 0};
    int status = 0;
    row[i >> 6] |= 1ull << (i & 63);
    if (i < ns) {
        int a = i;
        for (;;) {
            const int p = s_par[a];
            if (p < 0) {
                if (p < -1) status |= EAGLE2_STATUS_BAD_TREE;
                break;
            }
            if (p >= a) {  // parents precede children: also bounds the walk
                status |= EAGLE2_STATUS_BAD_TREE;
                break;
            }
            row[p >> 6] |= 1ull << (p & 63);
            a = p;
        }
    }
    for (int w = 0; w < W; ++w) mask_bits[((long long)b * m + i) * W + w] = row[w];
    pos_ids[(long long)b * m + i] = pos;
    if (mask_dense) {
        uint8_t* d = mask_dense + ((long long)b * m + i) * m;
        for (int j = 0; j < m; ++j) d[j] = (uint8_t)((row[j >> 6] >> (j & 63)) & 1ull);
    }
    return status;
}

// Values are compared as integer codes throughout (fp64 compares are slow on this part).  The
// ranking is a bitonic sort of (code, index) pairs, padded to a power of two with code 0, which
// sorts behind every real value.  With `frontier` given there is no ranking at all (the ablation
// without reranking, Section 5.2): the selection is every node the expansion phase selected, i.e.
// every node that is some node's parent plus the last step's frontier, lowest indices first.
__global__ void __launch_bounds__(kRerankThreads)
rerank_kernel(const int32_t* __restrict__ tree_token, const int32_t* __restrict__ tree_parent,
              const double* __restrict__ tree_value, const int32_t* __restrict__ frontier, int k, int N,
              int P, int m, int most, int32_t* __restrict__ sel_index, int32_t* __restrict__ sel_parent,
              int32_t* __restrict__ sel_token, int32_t* __restrict__ sel_depth,
              int32_t* __restrict__ n_sel, const int32_t* __restrict__ kv_len, uint64_t* __restrict__ mask_bits,
              uint8_t* __restrict__ mask_dense, int32_t* __restrict__ pos_ids, int32_t* d_status) {
    extern __shared__ __align__(16) unsigned char s_dyn[];
    __shared__ int32_t s_selpar[EAGLE2_MAX_M], s_seldep[EAGLE2_MAX_M];  // the selection, for the mask rows
    unsigned long long* s_code = reinterpret_cast<unsigned long long*>(s_dyn);  // [N] value codes
    unsigned long long* s_key = s_code + N;                                     // [P] sort keys
    int32_t* s_idx = reinterpret_cast<int32_t*>(s_key + P);                     // [P] sort payload
    int32_t* s_par = s_idx + P;                                                 // [N]
    int32_t* s_flat = s_par + N;                                                // [N] flat position or -1
    __shared__ int s_scan[kRerankThreads];

    chain_wait();
    chain_release();
    const int b = blockIdx.x, tid = threadIdx.x;
    const int32_t* tok = tree_token + (long long)b * N;
    const int32_t* par = tree_parent + (long long)b * N;
    const double* val = tree_value + (long long)b * N;
    int status = 0;

    for (int i = tid; i < N; i += kRerankThreads) {
        int p = par[i];
        if (p < -1 || p >= i) {
            status |= EAGLE2_STATUS_BAD_TREE;
            p = -1;
        }
        double v = val[i];
        if (v != v) {
            status |= EAGLE2_STATUS_NONFINITE_LOGIT;
            v = -INFINITY;
        }
        s_par[i] = p;
        s_code[i] = value_code(v);
        s_flat[i] = -1;
    }
    __syncthreads();
    if (frontier) {
        for (int i = tid; i < N; i += kRerankThreads)
            if (s_par[i] >= 0) s_flat[s_par[i]] = 0;  // several children store the same 0
        if (tid < k) {
            const int f = frontier[(long long)b * k + tid];
            if (f < 0 || f >= N) status |= EAGLE2_STATUS_BAD_TREE;
            else s_flat[f] = 0;
        }
    } else {
    // effective value = minimum of the values on the path from the root (parents have lower
    // indices, so the walk ends)
    for (int i = tid; i < P; i += kRerankThreads) {
        unsigned long long c = 0;
        if (i < N) {
            c = s_code[i];
            for (int a = s_par[i]; a >= 0; a = s_par[a]) c = s_code[a] < c ? s_code[a] : c;
        }
        s_key[i] = c;
        s_idx[i] = i;
    }
    __syncthreads();
    // order: effective value descending, index ascending
    if (P <= kRerankThreads) {
        // one element per thread (threads past P hold padding): exchanges closer than a warp go
        // through shuffles, the others through a double-buffered shared-memory copy
        __shared__ unsigned long long s_xk[2][kRerankThreads];
        __shared__ int32_t s_xi[2][kRerankThreads];
        unsigned long long key = tid < P ? s_key[tid] : 0ull;
        int idx = tid;
        int flip = 0;
#pragma unroll 1
        for (int size = 2; size <= kRerankThreads; size <<= 1) {
#pragma unroll 1
            for (int stride = size >> 1; stride > 0; stride >>= 1) {
                unsigned long long ok;
                int oi;
                if (stride < 32) {
                    ok = __shfl_xor_sync(0xffffffffu, key, stride);
                    oi = __shfl_xor_sync(0xffffffffu, idx, stride);
                } else {
                    s_xk[flip][tid] = key;
                    s_xi[flip][tid] = idx;
                    __syncthreads();
                    ok = s_xk[flip][tid ^ stride];
                    oi = s_xi[flip][tid ^ stride];
                    flip ^= 1;
                }
                const bool mine_first = key > ok || (key == ok && idx < oi);
                const bool keep_first = ((tid & stride) == 0) == ((tid & size) == 0);
                if (mine_first != keep_first) key = ok, idx = oi;
            }
        }
        if (tid < most) s_flat[idx] = 0;
    } else {
        for (int size = 2; size <= P; size <<= 1) {
            for (int stride = size >> 1; stride > 0; stride >>= 1) {
                for (int i = tid; i < P; i += kRerankThreads) {
                    const int j = i ^ stride;
                    if (j > i) {
                        const unsigned long long ki = s_key[i], kj = s_key[j];
                        const int ii = s_idx[i], ij = s_idx[j];
                        const bool i_first = ki > kj || (ki == kj && ii < ij);  // i belongs before j
                        const bool forward = (i & size) == 0;
                        if (i_first != forward) {
                            s_key[i] = kj, s_key[j] = ki;
                            s_idx[i] = ij, s_idx[j] = ii;
                        }
                    }
                }
                __syncthreads();
            }
        }
        for (int r = tid; r < most; r += kRerankThreads) s_flat[s_idx[r]] = 0;
    }
    }
    __syncthreads();
    // exclusive scan of the per-thread counts -> flat positions in ascending index
    const int per = (N + kRerankThreads - 1) / kRerankThreads;
    const int lo = min(N, tid * per), hi = min(N, lo + per);
    int mine = 0;
    for (int i = lo; i < hi; ++i) mine += s_flat[i] == 0;
    const int lane = tid & 31, warp = tid >> 5;
    int incl = mine;
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) {
        const int up = __shfl_up_sync(0xffffffffu, incl, o);
        if (lane >= o) incl += up;
    }
    if (lane == 31) s_scan[warp] = incl;
    __syncthreads();
    if (warp == 0) {
        int w = lane < kRerankThreads / 32 ? s_scan[lane] : 0;
#pragma unroll
        for (int o = 1; o < 32; o <<= 1) {
            const int up = __shfl_up_sync(0xffffffffu, w, o);
            if (lane >= o) w += up;
        }
        if (lane < kRerankThreads / 32) s_scan[lane] = w;  // inclusive totals of the warps
    }
    __syncthreads();
    int pos = incl - mine + (warp ? s_scan[warp - 1] : 0);
    const int keep = min(most, s_scan[kRerankThreads / 32 - 1]);  // fewer than `most` only without ranking
    for (int i = lo; i < hi; ++i)
        if (s_flat[i] == 0) {
            s_flat[i] = pos < most ? pos : -1;
            ++pos;
        }
    __syncthreads();

    int32_t* o_idx = sel_index + (long long)b * m;
    int32_t* o_par = sel_parent + (long long)b * m;
    int32_t* o_tok = sel_token + (long long)b * m;
    int32_t* o_dep = sel_depth + (long long)b * m;
    for (int i = tid; i < N; i += kRerankThreads) {
        const int j = s_flat[i];
        if (j < 0) continue;
        const int p = s_par[i];
        int fp = -1;
        if (p >= 0) {
            fp = s_flat[p];
            if (fp < 0) status |= EAGLE2_STATUS_NOT_CLOSED;
        }
        const int dep = i < k ? 0 : 1 + (i - k) / (k * k);
        o_idx[j] = i;
        o_par[j] = fp;
        o_tok[j] = tok[i];
        o_dep[j] = dep;
        s_selpar[j] = fp;
        s_seldep[j] = dep;
    }
    for (int j = keep + tid; j < m; j += kRerankThreads) {
        o_idx[j] = -1;
        o_par[j] = -1;
        o_tok[j] = 0;
        o_dep[j] = 0;
        s_selpar[j] = -1;
        s_seldep[j] = 0;
    }
    if (tid == 0) n_sel[b] = keep;
    if (mask_bits) {  // the mask rows and position ids of this selection, in the same launch
        __syncthreads();
        if (tid < m) status |= mask_row(s_selpar, tid, keep, m, b, kv_len[b] + (tid < keep ? s_seldep[tid] : 0), mask_bits,
                                        mask_dense, pos_ids);
    }
    if (status) raise_status(d_status, status);
}

__global__ void __launch_bounds__(EAGLE2_MAX_M)
tree_mask_kernel(const int32_t* __restrict__ sel_parent, const int32_t* __restrict__ sel_depth,
                 const int32_t* __restrict__ n_sel, const int32_t* __restrict__ kv_len, int m,
                 uint64_t* __restrict__ mask_bits, uint8_t* __restrict__ mask_dense,
                 int32_t* __restrict__ pos_ids, int32_t* d_status) {
    __shared__ int32_t s_par[EAGLE2_MAX_M];
    chain_wait();
    chain_release();
    const int b = blockIdx.x, i = threadIdx.x;
    const int ns = n_sel[b];
    if (i < m) s_par[i] = sel_parent[(long long)b * m + i];
    __syncthreads();
    if (i >= m) return;
    const int status = mask_row(s_par, i, ns, m, b, kv_len[b] + (i < ns ? sel_depth[(long long)b * m + i] : 0), mask_bits,
                                mask_dense, pos_ids);
    if (status) raise_status(d_status, status);
}

}  // namespace eagle2

using namespace eagle2;

// frontier == nullptr: the paper's reranking; else the selection the expansion phase made.
static int rerank_launch(const int32_t* tree_token, const int32_t* tree_parent, const double* tree_value,
                         const int32_t* frontier, int B, int k, int D, int m, int32_t* sel_index,
                         int32_t* sel_parent, int32_t* sel_token, int32_t* sel_depth, int32_t* n_sel,
                         const int32_t* kv_len, uint64_t* mask_bits, uint8_t* mask_dense, int32_t* pos_ids,
                         int32_t* d_status, eagle2_stream_t stream) {
    if (!tree_token || !tree_parent || !tree_value || !sel_index || !sel_parent || !sel_token ||
        !sel_depth || !n_sel || !d_status)
        return EAGLE2_ERR_NULL;
    if (B < 0 || k < 1 || k > EAGLE2_MAX_K || D < 1 || D > EAGLE2_MAX_DEPTH || m < 1 ||
        m > EAGLE2_MAX_M || nodes_of(k, D) > EAGLE2_MAX_NODES)
        return EAGLE2_ERR_SHAPE;
    if (!aligned(tree_value, 8)) return EAGLE2_ERR_ALIGN;
    if (B == 0) return EAGLE2_OK;
    const int N = (int)nodes_of(k, D);
    const int most = m < N ? m : N;
    int P = 1;
    while (P < N) P <<= 1;
    const size_t dyn = (size_t)N * (sizeof(unsigned long long) + 2 * sizeof(int32_t)) +
                       (size_t)P * (sizeof(unsigned long long) + sizeof(int32_t));
    if (dyn > 40 * 1024 &&
        cudaFuncSetAttribute(rerank_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)dyn) !=
            cudaSuccess)
        return EAGLE2_ERR_CUDA;
    return launch_chained(rerank_kernel, dim3(B), dim3(kRerankThreads), dyn, reinterpret_cast<cudaStream_t>(stream), 1,
                          tree_token, tree_parent, tree_value, frontier, k, N, P, m, most, sel_index, sel_parent,
                          sel_token, sel_depth, n_sel, kv_len, mask_bits, mask_dense, pos_ids, d_status);
}

extern "C" int eagle2_rerank(const int32_t* tree_token, const int32_t* tree_parent,
                             const double* tree_value, int B, int k, int D, int m, int32_t* sel_index,
                             int32_t* sel_parent, int32_t* sel_token, int32_t* sel_depth,
                             int32_t* n_sel, int32_t* d_status, eagle2_stream_t stream) {
    return rerank_launch(tree_token, tree_parent, tree_value, nullptr, B, k, D, m, sel_index, sel_parent,
                         sel_token, sel_depth, n_sel, nullptr, nullptr, nullptr, nullptr, d_status, stream);
}

extern "C" int eagle2_rerank_mask(const int32_t* tree_token, const int32_t* tree_parent, const double* tree_value,
                                  const int32_t* kv_len, int B, int k, int D, int m, int32_t* sel_index,
                                  int32_t* sel_parent, int32_t* sel_token, int32_t* sel_depth, int32_t* n_sel,
                                  uint64_t* mask_bits, uint8_t* mask_dense, int32_t* pos_ids, int32_t* d_status,
                                  eagle2_stream_t stream) {
    if (!kv_len || !mask_bits || !pos_ids) return EAGLE2_ERR_NULL;
    if (!aligned(mask_bits, 8)) return EAGLE2_ERR_ALIGN;
    return rerank_launch(tree_token, tree_parent, tree_value, nullptr, B, k, D, m, sel_index, sel_parent,
                         sel_token, sel_depth, n_sel, kv_len, mask_bits, mask_dense, pos_ids, d_status, stream);
}

extern "C" int eagle2_rerank_skipped(const int32_t* tree_token, const int32_t* tree_parent,
                                     const double* tree_value, const int32_t* frontier, int B, int k,
                                     int D, int m, int32_t* sel_index, int32_t* sel_parent,
                                     int32_t* sel_token, int32_t* sel_depth, int32_t* n_sel,
                                     int32_t* d_status, eagle2_stream_t stream) {
    if (!frontier) return EAGLE2_ERR_NULL;
    return rerank_launch(tree_token, tree_parent, tree_value, frontier, B, k, D, m, sel_index, sel_parent,
                         sel_token, sel_depth, n_sel, nullptr, nullptr, nullptr, nullptr, d_status, stream);
}

extern "C" int eagle2_tree_mask(const int32_t* sel_parent, const int32_t* sel_depth,
                                const int32_t* n_sel, const int32_t* kv_len, int B, int m,
                                uint64_t* mask_bits, uint8_t* mask_dense, int32_t* pos_ids,
                                int32_t* d_status, eagle2_stream_t stream) {
    if (!sel_parent || !sel_depth || !n_sel || !kv_len || !mask_bits || !pos_ids || !d_status)
        return EAGLE2_ERR_NULL;
    if (B < 0 || m < 1 || m > EAGLE2_MAX_M) return EAGLE2_ERR_SHAPE;
    if (!aligned(mask_bits, 8)) return EAGLE2_ERR_ALIGN;
    if (B == 0) return EAGLE2_OK;
    return launch_chained(tree_mask_kernel, dim3(B), dim3(EAGLE2_MAX_M), 0, reinterpret_cast<cudaStream_t>(stream), 1,
                          sel_parent, sel_depth, n_sel, kv_len, m, mask_bits, mask_dense, pos_ids, d_status);
}
