// Step 1 of the hot path: draft-tree expansion (paper Section 4.1).
//
// One launch per expansion step.  Block (chunk, row, sequence) holds a chunk of one logit row in
// registers, reduces it to (max, sum exp) and its k best tokens, and writes that partial to the
// workspace.  The last block of a sequence to arrive merges the partials of every row in fp64
// (log-sum-exp, top-k), writes the new tree level (token, parent, value = parent value + log-prob)
// and ranks the new candidates by value to produce the next frontier.
#include <math.h>

#include "vocab_scan.cuh"

namespace eagle2 {

struct ExpandPlan {
    int vpt;     // float4 per thread per chunk
    int chunks;  // chunks per row
};

constexpr int kMergeKeysMax = 3200;  // per-row partial keys the merging block can hold per warp

static bool expand_plan(long long rows, int V, int k, ExpandPlan* p) {
    int vpt = scan_pick_vpt(rows, V);
    while (vpt < 4 && (long long)scan_chunks(V, vpt) * k > kMergeKeysMax) vpt <<= 1;
    p->vpt = vpt;
    p->chunks = scan_chunks(V, vpt);
    return (long long)p->chunks * k <= kMergeKeysMax;
}

struct ExpandWs {
    int* counters;                  // [B] arrival tickets
    double2* stats;                 // [B][n_s][chunks] (max, sum exp(x - max))
    unsigned long long* keys;       // [B][n_s][chunks][k]
};

static size_t expand_ws_layout(int B, int n_s, int chunks, int k, void* base, ExpandWs* w) {
    size_t off = 0;
    char* p = static_cast<char*>(base);
    if (w) w->counters = reinterpret_cast<int*>(p + off);
    off += round_up(sizeof(int) * (size_t)B, kWsAlign);
    if (w) w->stats = reinterpret_cast<double2*>(p + off);
    off += round_up(sizeof(double2) * (size_t)B * n_s * chunks, kWsAlign);
    if (w) w->keys = reinterpret_cast<unsigned long long*>(p + off);
    off += round_up(sizeof(unsigned long long) * (size_t)B * n_s * chunks * k, kWsAlign);
    return off;
}

size_t expand_workspace_bytes(int B, int V, int k) {
    size_t need = 0;
    for (int n_s = 1; n_s <= k; n_s += (k > 1 ? k - 1 : 1)) {  // n_s = 1 and n_s = k
        ExpandPlan p;
        expand_plan((long long)B * n_s, V, k, &p);
        const size_t b = expand_ws_layout(B, n_s, p.chunks, k, nullptr, nullptr);
        need = b > need ? b : need;
    }
    return need;
}

template <int VPT, bool VEC>
__global__ void __launch_bounds__(kScanThreads)
expand_kernel(const float* __restrict__ draft_logits, long long batch_stride, int V, int k, int D,
              int s, int n_s, int chunks, int32_t* __restrict__ tree_token,
              int32_t* __restrict__ tree_parent, double* __restrict__ tree_value,
              int32_t* __restrict__ frontier, ExpandWs ws, int32_t* d_status) {
    constexpr int NE = 4 * VPT;
    __shared__ float s_redf[kScanWarps];
    __shared__ double s_redd[kScanWarps];
    __shared__ unsigned long long s_keys[kScanWarps * EAGLE2_MAX_K];
    __shared__ int s_flag;
    extern __shared__ __align__(16) unsigned char s_dyn[];

    const int chunk = blockIdx.x % chunks;
    const int row = (blockIdx.x / chunks) % n_s;
    const int b = blockIdx.x / (chunks * n_s);
    const float* zrow = draft_logits + (long long)b * batch_stride + (long long)row * V;

    // ---- scan this chunk -------------------------------------------------------------------
    float x[NE];
    scan_load<VPT, VEC>(zrow, V, chunk, x);
    float tmax = -INFINITY;
    int bad = 0;
#pragma unroll
    for (int j = 0; j < NE; ++j) {
        bad |= !(x[j] < INFINITY);  // NaN or +Inf
        tmax = fmaxf(tmax, x[j]);
    }
    const float cmax = block_max_f32(tmax, s_redf);
    float tsum = 0.f;
    if (cmax > -INFINITY) {
#pragma unroll
        for (int j = 0; j < NE; ++j) tsum += expf(x[j] - cmax);
    }
    const double csum = block_sum_f64((double)tsum, s_redd);
    unsigned long long key[NE];
#pragma unroll
    for (int j = 0; j < NE; ++j) {
        const int e = scan_elem_index<VPT, VEC>(chunk, j);
        key[j] = e < V ? make_key(x[j], (uint32_t)e) : 0ull;
    }
    const size_t part = ((size_t)b * n_s + row) * chunks + chunk;
    block_topk<NE>(key, k, s_keys, ws.keys + part * k);
    if (threadIdx.x == 0) ws.stats[part] = make_double2((double)cmax, csum);
    if (bad) raise_status(d_status, EAGLE2_STATUS_NONFINITE_LOGIT);

    // ---- the last block of this sequence merges ---------------------------------------------
    if (!last_block_arrives(ws.counters + b, chunks * n_s, &s_flag)) return;

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const long long N = nodes_of(k, D);
    const long long base = s ? (long long)k + (long long)(s - 1) * k * k : 0;
    const long long prev_base = s >= 2 ? (long long)k + (long long)(s - 2) * k * k : 0;
    const long long prev_count = s >= 2 ? (long long)k * k : k;
    const int n_new = n_s * k;
    const int keys_per_row = chunks * k;
    // dynamic shared memory: per-warp key staging, then the new candidates' values
    unsigned long long* s_stage = reinterpret_cast<unsigned long long*>(s_dyn) + (size_t)warp * keys_per_row;
    double* s_val = reinterpret_cast<double*>(reinterpret_cast<unsigned long long*>(s_dyn) +
                                              (size_t)kScanWarps * keys_per_row);
    int32_t* tok = tree_token + (long long)b * N;
    int32_t* par = tree_parent + (long long)b * N;
    double* val = tree_value + (long long)b * N;
    int32_t* fr = frontier + (long long)b * k;
    int status = 0;

    for (int r = warp; r < n_s; r += kScanWarps) {
        const size_t p0 = ((size_t)b * n_s + r) * chunks;
        // log-sum-exp of the row from the chunk partials, in double
        double m = -INFINITY;
        for (int c = lane; c < chunks; c += 32) m = fmax(m, ws.stats[p0 + c].x);
        m = warp_max_f64(m);
        double sum = 0.0;
        for (int c = lane; c < chunks; c += 32) {
            const double2 st = ws.stats[p0 + c];
            if (st.x > -INFINITY) sum += st.y * exp(st.x - m);
        }
        sum = warp_sum_f64(sum);
        if (!(m > -INFINITY)) status |= EAGLE2_STATUS_NONFINITE_LOGIT;
        const double lse = m + log(sum);
        // top-k of the chunk winners
        for (int e = lane; e < keys_per_row; e += 32) s_stage[e] = ws.keys[p0 * k + e];
        __syncwarp();
        int parent = -1;
        double parent_value = 0.0;
        if (s) {
            parent = fr[r];
            if (parent < prev_base || parent >= prev_base + prev_count) {
                status |= EAGLE2_STATUS_BAD_TREE;
                parent = (int)prev_base;
            }
            parent_value = val[parent];
        }
        for (int c = 0; c < k; ++c) {
            unsigned long long best = 0;
            for (int e = lane; e < keys_per_row; e += 32) best = s_stage[e] > best ? s_stage[e] : best;
            const unsigned long long top = warp_max_u64(best);
            for (int e = lane; e < keys_per_row; e += 32)
                if (s_stage[e] == top) s_stage[e] = 0ull;
            __syncwarp();
            if (lane == 0) {
                const long long node = base + (long long)r * k + c;
                const double v = parent_value + ((double)key_value(top) - lse);
                tok[node] = (int32_t)key_index(top);
                par[node] = parent;
                val[node] = v;
                s_val[r * k + c] = (v == v) ? v : -INFINITY;
            }
        }
    }
    __syncthreads();  // all rows merged; every read of the old frontier is done

    // next frontier: rank the new candidates by (value desc, index asc); ranks < k are kept
    for (int i = threadIdx.x; i < n_new; i += kScanThreads) {
        const double vi = s_val[i];
        int rank = 0;
        for (int j = 0; j < n_new; ++j) {
            const double vj = s_val[j];
            rank += (vj > vi) || (vj == vi && j < i);
        }
        if (rank < k) fr[rank] = (int32_t)(base + i);
    }
    if (status && lane == 0) raise_status(d_status, status);
}

template <int VPT, bool VEC>
static int launch_expand(const float* draft_logits, long long batch_stride, int B, int V, int k, int D,
                         int s, int n_s, int chunks, int32_t* tree_token, int32_t* tree_parent,
                         double* tree_value, int32_t* frontier, const ExpandWs& ws, int32_t* d_status,
                         cudaStream_t stream) {
    const size_t dyn = sizeof(unsigned long long) * (size_t)kScanWarps * chunks * k +
                       sizeof(double) * (size_t)n_s * k;
    auto kern = expand_kernel<VPT, VEC>;
    if (dyn > 40 * 1024 &&
        cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)dyn) != cudaSuccess)
        return EAGLE2_ERR_CUDA;
    const long long blocks = (long long)B * n_s * chunks;
    kern<<<(unsigned)blocks, kScanThreads, dyn, stream>>>(draft_logits, batch_stride, V, k, D, s, n_s,
                                                          chunks, tree_token, tree_parent, tree_value,
                                                          frontier, ws, d_status);
    return launch_result();
}

}  // namespace eagle2

using namespace eagle2;

extern "C" int eagle2_expand(const float* draft_logits, long long batch_stride, int B, int V, int k,
                             int D, int s, int32_t* tree_token, int32_t* tree_parent,
                             double* tree_value, int32_t* frontier, void* ws, size_t ws_bytes,
                             int32_t* d_status, eagle2_stream_t stream) {
    if (!draft_logits || !tree_token || !tree_parent || !tree_value || !frontier || !d_status)
        return EAGLE2_ERR_NULL;
    if (B < 0 || V < 1 || k < 1 || k > V || k > EAGLE2_MAX_K || D < 1 || D > EAGLE2_MAX_DEPTH || s < 0 ||
        s >= D || nodes_of(k, D) > EAGLE2_MAX_NODES || batch_stride < 0)
        return EAGLE2_ERR_SHAPE;
    if (!aligned(draft_logits, 4) || !aligned(tree_value, 8)) return EAGLE2_ERR_ALIGN;
    if (B == 0) return EAGLE2_OK;
    const int n_s = s ? k : 1;
    ExpandPlan plan;
    if (!expand_plan((long long)B * n_s, V, k, &plan)) return EAGLE2_ERR_SHAPE;
    if ((long long)B * n_s * plan.chunks > 0x7fffffffLL) return EAGLE2_ERR_SHAPE;
    if (!ws || !aligned(ws, kWsAlign)) return EAGLE2_ERR_WORKSPACE;
    ExpandWs w;
    if (expand_ws_layout(B, n_s, plan.chunks, k, ws, &w) > ws_bytes) return EAGLE2_ERR_WORKSPACE;
    const bool vec = aligned(draft_logits, 16) && V % 4 == 0 && batch_stride % 4 == 0;
    cudaStream_t st = reinterpret_cast<cudaStream_t>(stream);
#define EAGLE2_EXPAND_CASE(VPT_)                                                                      \
    case VPT_:                                                                                        \
        return vec ? launch_expand<VPT_, true>(draft_logits, batch_stride, B, V, k, D, s, n_s,        \
                                               plan.chunks, tree_token, tree_parent, tree_value,      \
                                               frontier, w, d_status, st)                             \
                   : launch_expand<VPT_, false>(draft_logits, batch_stride, B, V, k, D, s, n_s,       \
                                                plan.chunks, tree_token, tree_parent, tree_value,     \
                                                frontier, w, d_status, st);
    switch (plan.vpt) {
        EAGLE2_EXPAND_CASE(1)
        EAGLE2_EXPAND_CASE(2)
        EAGLE2_EXPAND_CASE(4)
    }
#undef EAGLE2_EXPAND_CASE
    return EAGLE2_ERR_SHAPE;
}
