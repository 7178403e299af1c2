// Step 1 of the hot path: draft-tree expansion (paper Section 4.1).
//
// One launch per expansion step.  Block (segment, row, sequence) streams its segment of one logit
// row in tiles of 4096 tokens (next tile's loads in flight while the current one is processed),
// keeps a per-thread running (max, sum exp) and a block list of top-k candidates filtered by the
// value of the block's k-th best so far, and writes one partial per segment to the workspace.  The
// last block of a sequence to arrive merges the partials, a warp per row (fp64 log-sum-exp, top-k of
// the segment winners), writes the new tree level (token, parent, value = parent value + log-prob)
// and ranks the new candidates by value to produce the next frontier.
#include <math.h>

#include <mutex>

#include "vocab_scan.cuh"

namespace eagle2 {

constexpr int kTileTokens = kScanThreads * 16;  // tokens per tile: four float4 per thread

struct ExpandPlan {
    int chunks;  // segments per row = blocks per row
    int tpb;     // tiles per block
};

constexpr int kMergeKeysMax = 1024;  // segment winners per row that the merge handles (32 per lane, two passes of 16)

// Enough blocks to fill the device three deep when the rows allow it, otherwise about 8 tiles per
// block; never more segments per row than the merge can take, whole tiles per segment.
static bool expand_plan(long long rows, int V, int k, ExpandPlan* p) {
    const int tiles = (V + kTileTokens - 1) / kTileTokens;
    long long g = (3 * 148 + rows - 1) / (rows > 0 ? rows : 1);
    if (g < (tiles + 7) / 8) g = (tiles + 7) / 8;  // at most 8 tiles per block: several waves balance out
    if (g > tiles) g = tiles;
    if (g * k > kMergeKeysMax) g = kMergeKeysMax / k;
    if (g < 1) g = 1;
    p->tpb = (int)((tiles + g - 1) / g);
    p->chunks = (tiles + p->tpb - 1) / p->tpb;
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

constexpr int kRing = 3;                                  // tiles in flight per block (vector path)
constexpr long long kExpandWaitCycles = 1LL << 31;       // ~1 s bound of a wait for a tile

__device__ __forceinline__ uint32_t smem_addr(const void* p) { return (uint32_t)__cvta_generic_to_shared(p); }
// one tile of a row, global -> shared, completion counted in bytes on an mbarrier
__device__ __forceinline__ void bulk_load(uint32_t dst, const void* src, uint32_t bytes, uint32_t bar) {
    asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(bar), "r"(bytes) : "memory");
    asm volatile("cp.async.bulk.shared::cta.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];"
                 ::"r"(dst), "l"(src), "r"(bytes), "r"(bar)
                 : "memory");
}
__device__ __forceinline__ bool tile_landed(uint32_t bar, uint32_t parity) {
    uint32_t ok;
    asm volatile(
        "{\n\t.reg .pred p;\n\tmbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\tselp.b32 %0, 1, 0, p;\n\t}"
        : "=r"(ok)
        : "r"(bar), "r"(parity)
        : "memory");
    return ok != 0;
}

__device__ __forceinline__ float fast_ex2(float x) {
    float y;
    asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
    return y;
}

template <bool VEC>
__global__ void __launch_bounds__(kScanThreads, 3)
expand_kernel(const float* __restrict__ draft_logits, long long batch_stride, int V, int k, int D,
              int s, int n_s, int chunks, int tpb, int32_t* __restrict__ tree_token,
              int32_t* __restrict__ tree_parent, double* __restrict__ tree_value,
              int32_t* __restrict__ frontier, ExpandWs ws, int32_t* d_status) {
    constexpr int VPT = 4, NE = 16;
    constexpr float kLog2e = 1.4426950408889634f;
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
    const int tiles = (V + kTileTokens - 1) / kTileTokens;
    const int t0 = chunk * tpb, t1 = min(tiles, t0 + tpb);

    // Vector path: tiles arrive by bulk copies into a ring in shared memory, kRing in flight.
    // Scalar path (unaligned rows): the next tile is prefetched into registers.
    extern __shared__ __align__(128) float s_ring[];  // [kRing][kTileTokens]
    __shared__ unsigned long long s_bar[kRing];
    auto issue_tile = [&](int t) {  // thread 0 only
        const int first = t * kTileTokens;
        const uint32_t bytes = (uint32_t)min(kTileTokens, V - first) * 4u;
        bulk_load(smem_addr(s_ring + (size_t)((t - t0) % kRing) * kTileTokens), zrow + first, bytes,
                  smem_addr(&s_bar[(t - t0) % kRing]));
    };
    if (VEC) {
        if (threadIdx.x == 0) {
            for (int i = 0; i < kRing; ++i)
                asm volatile("mbarrier.init.shared::cta.b64 [%0], 1;" ::"r"(smem_addr(&s_bar[i])) : "memory");
            asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
            for (int t = t0; t < t1 && t < t0 + kRing; ++t) issue_tile(t);
        }
    }
    float cur[NE], nxt[NE];
    if (!VEC) scan_load<VPT, false>(zrow, V, t0, cur);
    int timed_out = 0;
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
    if (threadIdx.x == 0) s_topk.count = 0, s_topk.overflow = 0, s_topk.thr = -INFINITY;
    for (int i = threadIdx.x; i < kCandCap; i += kScanThreads) s_topk.cand[i] = 0ull;  // empty list
    __syncthreads();  // also: the ring's barriers are initialised for every thread

    // ---- stream the segment ------------------------------------------------------------------------
    float m_t = -INFINITY, s_t = 0.f;  // this thread's running maximum and sum of exp(x - m_t)
    for (int t = t0; t < t1; ++t) {
        if (VEC) {
            const int slot = (t - t0) % kRing;
            const uint32_t parity = (uint32_t)(((t - t0) / kRing) & 1);
            const long long w0 = clock64();
            while (!tile_landed(smem_addr(&s_bar[slot]), parity)) {
                if (clock64() - w0 > kExpandWaitCycles) {
                    timed_out = 1;
                    break;
                }
            }
            const float* tile = s_ring + (size_t)slot * kTileTokens;
#pragma unroll
            for (int i = 0; i < VPT; ++i) {
                const int off = (i * kScanThreads + (int)threadIdx.x) * 4;  // as scan_elem_index<VPT, true>
                float4 v = make_float4(-INFINITY, -INFINITY, -INFINITY, -INFINITY);
                if (!timed_out && t * kTileTokens + off < V) v = *reinterpret_cast<const float4*>(tile + off);
                cur[4 * i + 0] = v.x, cur[4 * i + 1] = v.y, cur[4 * i + 2] = v.z, cur[4 * i + 3] = v.w;
            }
        } else if (t + 1 < t1) {
            scan_load<VPT, false>(zrow, V, t + 1, nxt);
        }
        float tm = -INFINITY;
#pragma unroll
        for (int j = 0; j < NE; ++j) tm = fmaxf(tm, cur[j]);
        if (tm > m_t) {
            s_t *= fast_ex2((m_t - tm) * kLog2e);  // 0 when nothing was summed yet
            m_t = tm;
        }
        if (m_t > -INFINITY) {
            const float neg = -m_t * kLog2e;
#pragma unroll
            for (int j = 0; j < NE; ++j) s_t += fast_ex2(fmaf(cur[j], kLog2e, neg));
        }
        // candidates: elements at or above the value of the block's k-th best so far (it changes only
        // in a compaction, between block-wide barriers); for the first tile each warp uses the k-th
        // largest of its lanes' maxima (at least k elements reach it)
        float thr = s_topk.thr;
        const bool first = t == t0;
        if (first) thr = __shfl_sync(0xffffffffu, warp_sort_desc_f32(tm), k - 1);
        int cnt = 0;
        if (tm >= thr) {
#pragma unroll
            for (int j = 0; j < NE; ++j) cnt += (cur[j] >= thr) && (scan_elem_index<VPT, VEC>(t, j) < V);
        }
        int crowded = 0;  // the list overflowed or passed half of its capacity
        if (__ballot_sync(0xffffffffu, cnt > 0)) {
            int incl = cnt;
#pragma unroll
            for (int o = 1; o < 32; o <<= 1) {
                const int up = __shfl_up_sync(0xffffffffu, incl, o);
                if (lane >= o) incl += up;
            }
            const int total = __shfl_sync(0xffffffffu, incl, 31);
            int base = 0;
            if (lane == 0) base = atomicAdd(&s_topk.count, total);
            base = __shfl_sync(0xffffffffu, base, 0);
            if (base + total <= kCandCap) {
                if (cnt) {
                    int pos = base + incl - cnt;
#pragma unroll
                    for (int j = 0; j < NE; ++j) {
                        const int e = scan_elem_index<VPT, VEC>(t, j);
                        if (cur[j] >= thr && e < V) s_topk.cand[pos++] = make_key(cur[j], (uint32_t)e);
                    }
                }
            } else if (lane == 0) {
                s_topk.overflow = 1;  // this warp's range of the list stays empty (zero keys)
            }
            crowded = base + total > kCandCap / 2;
        }
        const bool last = t + 1 == t1;
        // One barrier per tile: every thread has read its part of the ring slot, the appends are
        // done, and all threads agree on whether the list needs compacting.
        const bool compact = __syncthreads_or(crowded) || first || last;
        if (VEC && threadIdx.x == 0 && t + kRing < t1) issue_tile(t + kRing);  // refill the slot just read
        if (compact) {
            const int overflow = s_topk.overflow;  // stable: the next appends come after this branch's barrier
            if (overflow) {
                // more candidates than the list holds (heavily ordered input): rank this tile exactly
                unsigned long long key[NE];
#pragma unroll
                for (int j = 0; j < NE; ++j) {
                    const int e = scan_elem_index<VPT, VEC>(t, j);
                    key[j] = e < V ? make_key(cur[j], (uint32_t)e) : 0ull;
                }
                block_topk<NE>(key, k, s_topk.exact, s_topk.win);
                __syncthreads();
            }
            if (warp == 0) {
                // best k of the list; after an overflow, of (the list without this tile's entries | the
                // tile's exact winners)
                const int n = min(s_topk.count, kCandCap);
                const uint32_t tile_first = (uint32_t)t * kTileTokens;
                unsigned long long mine[kCandCap / 32 + 1];
#pragma unroll
                for (int u = 0; u < kCandCap / 32; ++u) {
                    unsigned long long key = lane + 32 * u < n ? s_topk.cand[lane + 32 * u] : 0ull;
                    if (overflow && key && key_index(key) - tile_first < (uint32_t)kTileTokens) key = 0ull;
                    mine[u] = key;
                }
                mine[kCandCap / 32] = (overflow && lane < k) ? s_topk.win[lane] : 0ull;
                __syncwarp();
                warp_select<kCandCap / 32 + 1>(mine, k, s_topk.cand);
                __syncwarp();
                // past the k winners the list is empty again
#pragma unroll
                for (int u = 0; u < kCandCap / 32; ++u)
                    if (lane + 32 * u >= k && lane + 32 * u < n) s_topk.cand[lane + 32 * u] = 0ull;
                if (lane == 0) {
                    s_topk.count = k;  // entries past the keys that exist are 0 and never win
                    s_topk.overflow = 0;
                    s_topk.thr = s_topk.cand[k - 1] ? key_value(s_topk.cand[k - 1]) : -INFINITY;
                }
            }
            __syncthreads();
        }
        if (!VEC) {
#pragma unroll
            for (int j = 0; j < NE; ++j) cur[j] = nxt[j];
        }
    }
    if (timed_out) raise_status(d_status, EAGLE2_STATUS_TIMEOUT);

    // ---- the segment's partial: k best keys, (max, sum exp) ----------------------------------------
    const size_t part = ((size_t)b * n_s + row) * chunks + chunk;
    if (threadIdx.x < k) ws.keys[part * k + threadIdx.x] = s_topk.cand[threadIdx.x];
    const float wmax = warp_max_f32(m_t);
    float scaled = m_t > -INFINITY ? s_t * fast_ex2((m_t - wmax) * kLog2e) : 0.f;
    scaled = warp_sum_f32(scaled);
    if (lane == 0) s_wmax[warp] = wmax, s_wsum[warp] = scaled;
    int bad = !(scaled == scaled) || wmax == INFINITY;  // a NaN or +Inf logit poisons the sum / the max
    __syncthreads();
    if (threadIdx.x == 0) {
        float cmax = s_wmax[0];
#pragma unroll
        for (int w = 1; w < kScanWarps; ++w) cmax = fmaxf(cmax, s_wmax[w]);
        double csum = 0.0;
        if (cmax > -INFINITY) {
#pragma unroll
            for (int w = 0; w < kScanWarps; ++w)
                if (s_wmax[w] > -INFINITY) csum += (double)s_wsum[w] * exp((double)s_wmax[w] - (double)cmax);
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

template <bool VEC>
static int launch_expand(const float* draft_logits, long long batch_stride, int B, int V, int k, int D,
                         int s, int n_s, const ExpandPlan& plan, int32_t* tree_token, int32_t* tree_parent,
                         double* tree_value, int32_t* frontier, const ExpandWs& ws, int32_t* d_status,
                         cudaStream_t stream) {
    const long long blocks = (long long)B * n_s * plan.chunks;
    const size_t dyn = VEC ? sizeof(float) * (size_t)kRing * kTileTokens : 0;
    if (dyn > 40 * 1024 && cudaFuncSetAttribute(expand_kernel<VEC>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                                (int)dyn) != cudaSuccess) {
        cudaGetLastError();
        return EAGLE2_ERR_CUDA;
    }
    return launch_chained(expand_kernel<VEC>, dim3((unsigned)blocks), dim3(kScanThreads), dyn, stream, 1, draft_logits,
                          batch_stride, V, k, D, s, n_s, plan.chunks, plan.tpb, tree_token, tree_parent, tree_value,
                          frontier, ws, d_status);
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
    return vec ? launch_expand<true>(draft_logits, batch_stride, B, V, k, D, s, n_s, plan, tree_token, tree_parent,
                                     tree_value, frontier, w, d_status, st)
               : launch_expand<false>(draft_logits, batch_stride, B, V, k, D, s, n_s, plan, tree_token, tree_parent,
                                      tree_value, frontier, w, d_status, st);
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
    return vec ? launch_expand<true>(draft_logits, batch_stride, B, V, k, D, s, n_s, plan, tree_token, tree_parent,
                                     tree_value, frontier, w, d_status, st)
               : launch_expand<false>(draft_logits, batch_stride, B, V, k, D, s, n_s, plan, tree_token, tree_parent,
                                      tree_value, frontier, w, d_status, st);
}
