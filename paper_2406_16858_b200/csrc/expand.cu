// Step 1 of the hot path: draft-tree expansion (paper Section 4.1).
//
// One launch per expansion step.  Block (chunk, row, sequence) holds a chunk of one logit row in
// registers, reduces it to (max, sum exp) and its k best tokens, and writes that partial to the
// workspace.  The last block of a sequence to arrive merges the partials, a warp per row (fp64
// log-sum-exp, top-k of the chunk winners), writes the new tree level (token, parent, value = parent
// value + log-prob) and ranks the new candidates by value to produce the next frontier.
#include <math.h>

#include <mutex>

#include "vocab_scan.cuh"

namespace eagle2 {

struct ExpandPlan {
    int vpt;     // float4 per thread per chunk
    int chunks;  // chunks per row
};

constexpr int kMergeKeysMax = 1024;  // chunk winners per row that the merging warp holds in registers (32 per lane)

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
    off += counters_bytes(B);
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

// Monotone map double -> uint64 (larger value, larger code; -0 folded onto +0; NaN lowest).
__device__ __forceinline__ unsigned long long order_code_f64(double x) {
    if (x != x) return 0ull;
    const unsigned long long u = (unsigned long long)__double_as_longlong(x + 0.0);
    return (u >> 63) ? ~u : (u | 0x8000000000000000ull);
}

template <int VPT, bool VEC>
__global__ void __launch_bounds__(kScanThreads, 3)
expand_kernel(const float* __restrict__ draft_logits, long long batch_stride, int V, int k, int D,
              int s, int n_s, int chunks, int32_t* __restrict__ tree_token,
              int32_t* __restrict__ tree_parent, double* __restrict__ tree_value,
              int32_t* __restrict__ frontier, ExpandWs ws, int32_t* d_status) {
    constexpr int NE = 4 * VPT;
    __shared__ TopkScratch s_topk;
    __shared__ float s_wmax[kScanWarps], s_wsum[kScanWarps];
    __shared__ int s_flag;
    __shared__ unsigned long long s_rank[EAGLE2_MAX_K * EAGLE2_MAX_K];  // the new candidates' value codes

    chain_wait();
    chain_release();
    const int chunk = blockIdx.x % chunks;
    const int row = (blockIdx.x / chunks) % n_s;
    const int b = blockIdx.x / (chunks * n_s);
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const float* zrow = draft_logits + (long long)b * batch_stride + (long long)row * V;

    // ---- scan this chunk: per-warp (max, sum of exponentials), block top-k -----------------------
    float x[NE];
    scan_load<VPT, VEC>(zrow, V, chunk, x);
    // The block that arrives last merges every row and then needs the rows' parents and their
    // values; whichever block that will be, the two dependent loads are already under way.
    const long long N = nodes_of(k, D);
    int my_parent = -1;
    double my_parent_value = 0.0;
    if (s && threadIdx.x < n_s) {
        my_parent = frontier[(long long)b * k + threadIdx.x];
        const long long prev_base = s >= 2 ? (long long)k + (long long)(s - 2) * k * k : 0;
        const long long prev_count = s >= 2 ? (long long)k * k : k;
        if (my_parent < prev_base || my_parent >= prev_base + prev_count) my_parent = -2;  // reported by the merger
        else my_parent_value = tree_value[(long long)b * N + my_parent];
    }
    if (threadIdx.x == 0) s_topk.count = 0, s_topk.overflow = 0;
    float tmax = -INFINITY;
    int bad = 0;
#pragma unroll
    for (int j = 0; j < NE; ++j) {
        bad |= !(x[j] < INFINITY);  // NaN or +Inf
        tmax = fmaxf(tmax, x[j]);
    }
    const float wmax = warp_max_f32(tmax);
    float tsum = 0.f;
    if (wmax > -INFINITY) {
#pragma unroll
        for (int j = 0; j < NE; ++j) tsum += expf(x[j] - wmax);
    }
    tsum = warp_sum_f32(tsum);
    if (lane == 0) s_wmax[warp] = wmax, s_wsum[warp] = tsum;
    __syncthreads();
    const size_t part = ((size_t)b * n_s + row) * chunks + chunk;
    block_topk_filtered<VPT, VEC>(x, chunk, V, k, &s_topk, ws.keys + part * k);
    if (threadIdx.x == 0) {
        float cmax = s_wmax[0];
#pragma unroll
        for (int w = 1; w < kScanWarps; ++w) cmax = fmaxf(cmax, s_wmax[w]);
        double csum = 0.0;
        if (cmax > -INFINITY) {
#pragma unroll
            for (int w = 0; w < kScanWarps; ++w)
                if (s_wmax[w] > -INFINITY) csum += (double)s_wsum[w] * (double)expf(s_wmax[w] - cmax);
        }
        ws.stats[part] = make_double2((double)cmax, csum);
    }
    if (bad) raise_status(d_status, EAGLE2_STATUS_NONFINITE_LOGIT);

    // ---- the last block of this sequence merges: a warp per row -------------------------------
    if (!last_block_arrives(ws.counters + b, chunks * n_s, &s_flag)) return;

    __shared__ int s_parent[EAGLE2_MAX_K];
    __shared__ double s_pvalue[EAGLE2_MAX_K];
    const long long base = s ? (long long)k + (long long)(s - 1) * k * k : 0;
    const int n_new = n_s * k;
    const int keys_per_row = chunks * k;
    int32_t* tok = tree_token + (long long)b * N;
    int32_t* par = tree_parent + (long long)b * N;
    double* val = tree_value + (long long)b * N;
    int32_t* fr = frontier + (long long)b * k;
    if (threadIdx.x < n_s) s_parent[threadIdx.x] = my_parent, s_pvalue[threadIdx.x] = my_parent_value;
    __syncthreads();
    int status = 0;

    for (int r = warp; r < n_s; r += kScanWarps) {
        const size_t p0 = ((size_t)b * n_s + r) * chunks;
        constexpr int BATCH = 16;  // chunk winners per lane and pass
        // everything the row needs is requested before any of it is used
        unsigned long long cand[BATCH + 1];
#pragma unroll
        for (int t = 0; t < BATCH; ++t)
            cand[t] = lane + 32 * t < keys_per_row ? ws.keys[p0 * k + lane + 32 * t] : 0ull;
        double2 st0 = make_double2(-INFINITY, 0.0);
        if (lane < chunks) st0 = ws.stats[p0 + lane];
        int parent = s ? s_parent[r] : -1;
        const double parent_value = s ? s_pvalue[r] : 0.0;
        if (parent < -1) {
            status |= EAGLE2_STATUS_BAD_TREE;
            parent = (int)(s >= 2 ? (long long)k + (long long)(s - 2) * k * k : 0);
        }
        // log-sum-exp of the row from the chunk partials, in double
        double m = st0.x;
        for (int c = lane + 32; c < chunks; c += 32) m = fmax(m, ws.stats[p0 + c].x);
        m = warp_max_f64(m);
        double sum = st0.x > -INFINITY ? st0.y * exp(st0.x - m) : 0.0;
        for (int c = lane + 32; c < chunks; c += 32) {
            const double2 st = ws.stats[p0 + c];
            if (st.x > -INFINITY) sum += st.y * exp(st.x - m);
        }
        sum = warp_sum_f64(sum);
        if (!(m > -INFINITY)) status |= EAGLE2_STATUS_NONFINITE_LOGIT;
        const double lse = m + log(sum);
        // top-k of the chunk winners, 32*BATCH at a time together with the best so far; lane c ends
        // up holding the c-th.  The k-th largest lane maximum is a threshold no winner can be below;
        // when at most 32 keys reach it (the usual case) they are sorted across the lanes, otherwise
        // k rounds of maximum extraction do the same job.
        unsigned long long* s_pack = s_topk.cand + warp * 32;  // free: the chunk scan is over
        unsigned long long mine = 0;
        for (int e0 = 0; e0 < keys_per_row; e0 += 32 * BATCH) {
            if (e0) {
#pragma unroll
                for (int t = 0; t < BATCH; ++t)
                    cand[t] = e0 + lane + 32 * t < keys_per_row ? ws.keys[p0 * k + e0 + lane + 32 * t] : 0ull;
            }
            cand[BATCH] = mine;
            unsigned long long lane_best = 0;
#pragma unroll
            for (int t = 0; t <= BATCH; ++t) lane_best = cand[t] > lane_best ? cand[t] : lane_best;
            const unsigned long long thr = __shfl_sync(0xffffffffu, warp_sort_desc_u64(lane_best), k - 1);
            int cnt = 0;
#pragma unroll
            for (int t = 0; t <= BATCH; ++t) cnt += cand[t] >= thr && cand[t] != 0ull;
            int incl = cnt;
#pragma unroll
            for (int o = 1; o < 32; o <<= 1) {
                const int up = __shfl_up_sync(0xffffffffu, incl, o);
                if (lane >= o) incl += up;
            }
            const int total = __shfl_sync(0xffffffffu, incl, 31);
            unsigned long long next = 0;
            if (total <= 32) {
                int pos = incl - cnt;
#pragma unroll
                for (int t = 0; t <= BATCH; ++t)
                    if (cand[t] >= thr && cand[t] != 0ull) s_pack[pos++] = cand[t];
                __syncwarp();
                next = warp_sort_desc_u64(lane < total ? s_pack[lane] : 0ull);
                __syncwarp();
                if (lane >= k) next = 0ull;
            } else {
                for (int c = 0; c < k; ++c) {
                    unsigned long long best = 0;
#pragma unroll
                    for (int t = 0; t <= BATCH; ++t) best = cand[t] > best ? cand[t] : best;
                    const unsigned long long top = warp_max_u64(best);
#pragma unroll
                    for (int t = 0; t <= BATCH; ++t) cand[t] = (cand[t] == top) ? 0ull : cand[t];
                    if (lane == c) next = top;
                }
            }
            mine = next;
        }
        if (lane < k) {
            const long long node = base + (long long)r * k + lane;
            const double v = parent_value + ((double)key_value(mine) - lse);
            tok[node] = (int32_t)key_index(mine);
            par[node] = parent;
            val[node] = v;
            s_rank[r * k + lane] = order_code_f64(v);
        }
    }
    __syncthreads();  // all rows merged (the old frontier was read when the kernel started)

    // next frontier: rank the new candidates by (value desc, index asc); ranks < k are kept
    for (int i = threadIdx.x; i < n_new; i += kScanThreads) {
        const unsigned long long ci = s_rank[i];
        int rank = 0;
        for (int j = 0; j < n_new; ++j) {
            const unsigned long long cj = s_rank[j];
            rank += (cj > ci) || (cj == ci && j < i);
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
    auto kern = expand_kernel<VPT, VEC>;
    const long long blocks = (long long)B * n_s * chunks;
    return launch_chained(kern, dim3((unsigned)blocks), dim3(kScanThreads), 0, stream, 1, draft_logits, batch_stride, V,
                          k, D, s, n_s, chunks, tree_token, tree_parent, tree_value, frontier, ws, d_status);
}

// Scratch of eagle2_expand_static: lives in every context that loads the library, until exit.
static __device__ __align__(256) unsigned char g_expand_scratch[EAGLE2_EXPAND_STATIC_BYTES];

// Device address of g_expand_scratch on the current device (looked up once per device; in host
// code the array's name is only a handle for this query, never an address a kernel can use).
static int expand_scratch_address(void** out) {
    constexpr int kMaxDevices = 64;
    static void* addr[kMaxDevices] = {nullptr};
    static std::mutex mu;
    int dev = -1;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= kMaxDevices) {
        cudaGetLastError();
        return EAGLE2_ERR_CUDA;
    }
    std::lock_guard<std::mutex> lock(mu);
    if (!addr[dev]) {
        void* p = nullptr;
        if (cudaGetSymbolAddress(&p, g_expand_scratch) != cudaSuccess || !p) {
            cudaGetLastError();
            return EAGLE2_ERR_CUDA;
        }
        addr[dev] = p;
    }
    *out = addr[dev];
    return EAGLE2_OK;
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

extern "C" int eagle2_expand_static(const float* draft_logits, long long batch_stride, int B, int V, int k,
                                    int D, int s, int32_t* tree_token, int32_t* tree_parent,
                                    double* tree_value, int32_t* frontier, int32_t* d_status,
                                    eagle2_stream_t stream) {
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
    if (expand_ws_layout(B, n_s, plan.chunks, k, nullptr, nullptr) > (size_t)EAGLE2_EXPAND_STATIC_BYTES)
        return EAGLE2_ERR_STATIC_LIMIT;
    void* scratch = nullptr;
    const int rc = expand_scratch_address(&scratch);
    if (rc != EAGLE2_OK) return rc;
    ExpandWs w;
    expand_ws_layout(B, n_s, plan.chunks, k, scratch, &w);
    cudaStream_t st = reinterpret_cast<cudaStream_t>(stream);
    // the array keeps whatever the last call left: the arrival counters must start at zero
    if (cudaMemsetAsync(w.counters, 0, counters_bytes(B), st) != cudaSuccess) {
        cudaGetLastError();
        return EAGLE2_ERR_CUDA;
    }
    const bool vec = aligned(draft_logits, 16) && V % 4 == 0 && batch_stride % 4 == 0;
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
