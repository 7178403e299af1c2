// Step 1 of the hot path: draft-tree expansion (paper Section 4.1).
//
// One launch per expansion step.  Block (segment, row, sequence) streams its segment of one logit
// row in tiles of 4096 tokens (two tiles of asynchronous copies in flight ahead of the one being processed); each
// warp keeps per-thread running (max, sum exp) and its own short list of top-k candidates, and the
// block writes one partial per segment to the workspace.  The
// last block of a sequence to arrive merges the partials, a warp per row (fp64 log-sum-exp, top-k of
// the segment winners), writes the new tree level (token, parent, value = parent value + log-prob)
// and ranks the new candidates by value to produce the next frontier.
#include <math.h>

#include <mutex>
#include <type_traits>

#include "vocab_scan.cuh"

namespace eagle2 {

constexpr int kTileTokens = kScanThreads * 16;  // tokens per tile: four float4 per thread

struct ExpandPlan {
    int chunks;  // segments per row = blocks per row
    int tpb;     // tiles per block
};

constexpr int kMergeKeysMax = 1024;  // segment winners per row that the merge handles (32 per lane, two passes of 16)

// Segments per row.  A launch of up to three waves of one-tile blocks is about latency: one tile
// per block.  Otherwise a block costs about kBlockFixed tile times of start-up and hand-over on top
// of its tiles, an SM holds three blocks at once, and the choice minimises (rounds of resident blocks)
// x (cost of a block): measured per call at 320 rows of 128256 logits, 1 / 2 / 3 / 4 segments per row
// 54.7 / 63.4 / 71.1 / 76.1 us; at 80 rows the choice hardly matters (38-39 us for 2..8 segments).  Never more segments per row than the merge can take, whole tiles per
// segment.
static bool expand_plan(long long rows, int V, int k, ExpandPlan* p) {
    constexpr int kBlockFixed = 6;
    constexpr int kResident = 3;  // streaming blocks an SM holds at once (shared memory, launch bounds)
    const long long kSMs = sm_count();
    const int tiles = (V + kTileTokens - 1) / kTileTokens;
    long long g_max = kMergeKeysMax / k;
    if (g_max > tiles) g_max = tiles;
    if (g_max < 1) g_max = 1;
    if (rows < 1) rows = 1;
    long long g = g_max;
    if (rows * tiles > 9 * kSMs) {
        long long best = -1;
        for (long long c = 1; c <= g_max; ++c) {
            const long long tpb = (tiles + c - 1) / c;
            const long long cost = ((rows * c + kResident * kSMs - 1) / (kResident * kSMs)) * (kBlockFixed + tpb);
            if (best < 0 || cost < best) best = cost, g = c;
        }
    }
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

constexpr int kWarpList = 64;  // candidate keys a warp holds between two tightenings of its threshold

__device__ __forceinline__ float fast_ex2(float x) {
    float y;
    asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
    return y;
}

constexpr int kDepth = 3;  // tiles of a warp's ring: the one being read and two in flight

__device__ __forceinline__ uint32_t smem_addr(const void* p) { return (uint32_t)__cvta_generic_to_shared(p); }
__device__ __forceinline__ void async_copy16(uint32_t dst_shared, const float* src) {
    asm volatile("cp.async.cg.shared.global [%0], [%1], 16;" ::"r"(dst_shared), "l"(src) : "memory");
}
__device__ __forceinline__ void async_commit() { asm volatile("cp.async.commit_group;" ::: "memory"); }
template <int PENDING>
__device__ __forceinline__ void async_wait() {
    asm volatile("cp.async.wait_group %0;" ::"n"(PENDING) : "memory");
}

// warp_sort_desc_u64 for N independent keys per lane (key n of all lanes is one sequence): the N
// chains of dependent shuffles advance side by side.
template <int N>
__device__ __forceinline__ void warp_sort_desc_u64_n(unsigned long long (&v)[N]) {
    const int lane = threadIdx.x & 31;
#pragma unroll
    for (int size = 2; size <= 32; size <<= 1) {
#pragma unroll
        for (int stride = size >> 1; stride > 0; stride >>= 1) {
            const bool desc = (lane & size) == 0, lower = (lane & stride) == 0;
#pragma unroll
            for (int n = 0; n < N; ++n) {
                const unsigned long long other = __shfl_xor_sync(0xffffffffu, v[n], stride);
                const unsigned long long hi = v[n] > other ? v[n] : other, lo = v[n] > other ? other : v[n];
                v[n] = (lower == desc) ? hi : lo;
            }
        }
    }
}

constexpr int kQueue = 256;                              // candidate keys in flight to the selector warp

// Sorts a bitonic sequence of one key per lane (first rising then falling, or the reverse) into
// descending order.
__device__ __forceinline__ unsigned long long warp_bitonic_merge_desc(unsigned long long v) {
    const int lane = threadIdx.x & 31;
#pragma unroll
    for (int stride = 16; stride > 0; stride >>= 1) {
        const unsigned long long other = __shfl_xor_sync(0xffffffffu, v, stride);
        const unsigned long long hi = v > other ? v : other, lo = v > other ? other : v;
        v = (lane & stride) == 0 ? hi : lo;
    }
    return v;
}

// What the block that arrives last for a sequence does, a warp per row: the rows' log-sum-exp from
// the segments' statistics (fp64), the k best of the segments' winners, the new tree level (token,
// parent, value = parent value + log-probability) and the next frontier, ranked by value.  Also the
// whole of a merge-only launch, whose partials another kernel wrote in the same layout.
// my_parent / my_parent_value: thread r < n_s holds frontier slot r's node and its value.
__device__ __forceinline__ void expand_finish(int b, int V, int k, int D, int s, int n_s, int chunks, int by_confidence,
                                              int my_parent, double my_parent_value, int32_t* __restrict__ tree_token,
                                              int32_t* __restrict__ tree_parent, double* __restrict__ tree_value,
                                              int32_t* __restrict__ frontier, const ExpandWs& ws,
                                              unsigned long long (*s_list)[kWarpList], unsigned long long* s_rank,
                                              int32_t* d_status) {
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const long long N = nodes_of(k, D);
    (void)V;
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

    // A warp merges NR rows at a time, r and r + 8: the work of a row is a chain of dependent
    // shuffles, so when there are more rows than warps (the ten rows of a step on eight warps) the
    // second row rides along in the first one's latency instead of taking a second pass.
    auto merge_rows = [&](auto nr_tag, auto batch_tag) {
        constexpr int NR = decltype(nr_tag)::value;
        constexpr int BATCH = decltype(batch_tag)::value;  // chunk winners per lane and pass
        for (int r_base = warp; r_base < n_s; r_base += kScanWarps * NR) {
            int r[NR];
            bool valid[NR];
            size_t p0[NR];
            unsigned long long cand[NR][BATCH + 1];
            double2 st0[NR];
            int parent[NR];
            double parent_value[NR], lse[NR];
            // everything the rows need is requested before any of it is used
#pragma unroll
            for (int q = 0; q < NR; ++q) {
                r[q] = r_base + q * kScanWarps;
                valid[q] = r[q] < n_s;
                p0[q] = ((size_t)b * n_s + (valid[q] ? r[q] : 0)) * chunks;
#pragma unroll
                for (int t = 0; t < BATCH; ++t)
                    cand[q][t] = (valid[q] && lane + 32 * t < keys_per_row) ? ws.keys[p0[q] * k + lane + 32 * t] : 0ull;
                st0[q] = make_double2(-INFINITY, 0.0);
                if (valid[q] && lane < chunks) st0[q] = ws.stats[p0[q] + lane];
                parent[q] = (s && valid[q]) ? s_parent[r[q]] : -1;
                parent_value[q] = (s && valid[q]) ? s_pvalue[r[q]] : 0.0;
                if (parent[q] < -1) {
                    status |= EAGLE2_STATUS_BAD_TREE;
                    parent[q] = (int)(s >= 2 ? (long long)k + (long long)(s - 2) * k * k : 0);
                }
            }
            // log-sum-exp of the rows from the chunk partials, in double
#pragma unroll
            for (int q = 0; q < NR; ++q) {
                double m = st0[q].x;
                if (valid[q])
                    for (int c = lane + 32; c < chunks; c += 32) m = fmax(m, ws.stats[p0[q] + c].x);
                m = warp_max_f64(m);
                double sum = st0[q].x > -INFINITY ? st0[q].y * exp(st0[q].x - m) : 0.0;
                if (valid[q])
                    for (int c = lane + 32; c < chunks; c += 32) {
                        const double2 st = ws.stats[p0[q] + c];
                        if (st.x > -INFINITY) sum += st.y * exp(st.x - m);
                    }
                sum = warp_sum_f64(sum);
                if (valid[q] && !(m > -INFINITY)) status |= EAGLE2_STATUS_NONFINITE_LOGIT;
                lse[q] = m + log(sum);
            }
            // top-k of the chunk winners, 32*BATCH at a time together with the best so far; lane c ends
            // up holding the c-th.  The k-th largest lane maximum is a threshold no winner can be below;
            // when at most 32 keys reach it (the usual case) they are sorted across the lanes, otherwise
            // k rounds of maximum extraction do the same job.
            unsigned long long mine[NR];
#pragma unroll
            for (int q = 0; q < NR; ++q) mine[q] = 0ull;
            for (int e0 = 0; e0 < keys_per_row; e0 += 32 * BATCH) {
                unsigned long long thr[NR];
                int cnt[NR], incl[NR], total[NR];
#pragma unroll
                for (int q = 0; q < NR; ++q) {
                    if (e0) {
#pragma unroll
                        for (int t = 0; t < BATCH; ++t)
                            cand[q][t] = (valid[q] && e0 + lane + 32 * t < keys_per_row)
                                             ? ws.keys[p0[q] * k + e0 + lane + 32 * t]
                                             : 0ull;
                    }
                    cand[q][BATCH] = mine[q];
                }
                unsigned long long lane_best[NR];
#pragma unroll
                for (int q = 0; q < NR; ++q) {
                    lane_best[q] = 0;
#pragma unroll
                    for (int t = 0; t <= BATCH; ++t) lane_best[q] = cand[q][t] > lane_best[q] ? cand[q][t] : lane_best[q];
                }
                warp_sort_desc_u64_n<NR>(lane_best);
#pragma unroll
                for (int q = 0; q < NR; ++q) {
                    thr[q] = __shfl_sync(0xffffffffu, lane_best[q], k - 1);
                    cnt[q] = 0;
#pragma unroll
                    for (int t = 0; t <= BATCH; ++t) cnt[q] += cand[q][t] >= thr[q] && cand[q][t] != 0ull;
                    incl[q] = cnt[q];
                }
#pragma unroll
                for (int o = 1; o < 32; o <<= 1) {
#pragma unroll
                    for (int q = 0; q < NR; ++q) {
                        const int up = __shfl_up_sync(0xffffffffu, incl[q], o);
                        if (lane >= o) incl[q] += up;
                    }
                }
                bool packed = true;
                unsigned long long next[NR];
#pragma unroll
                for (int q = 0; q < NR; ++q) {
                    total[q] = __shfl_sync(0xffffffffu, incl[q], 31);
                    packed = packed && total[q] <= 32;
                    next[q] = 0ull;
                }
                if (packed) {  // every row of the warp: pack, then sort the rows side by side
#pragma unroll
                    for (int q = 0; q < NR; ++q) {
                        unsigned long long* s_pack = s_list[warp] + q * 32;  // free: the segment scan is over
                        int pos = incl[q] - cnt[q];
#pragma unroll
                        for (int t = 0; t <= BATCH; ++t)
                            if (cand[q][t] >= thr[q] && cand[q][t] != 0ull) s_pack[pos++] = cand[q][t];
                    }
                    __syncwarp();
#pragma unroll
                    for (int q = 0; q < NR; ++q) next[q] = lane < total[q] ? s_list[warp][q * 32 + lane] : 0ull;
                    warp_sort_desc_u64_n<NR>(next);
                    __syncwarp();
#pragma unroll
                    for (int q = 0; q < NR; ++q)
                        if (lane >= k) next[q] = 0ull;
                } else {
#pragma unroll
                    for (int q = 0; q < NR; ++q) {
                        for (int c = 0; c < k; ++c) {
                            unsigned long long best = 0;
#pragma unroll
                            for (int t = 0; t <= BATCH; ++t) best = cand[q][t] > best ? cand[q][t] : best;
                            const unsigned long long top = warp_max_u64(best);
#pragma unroll
                            for (int t = 0; t <= BATCH; ++t) cand[q][t] = (cand[q][t] == top) ? 0ull : cand[q][t];
                            if (lane == c) next[q] = top;
                        }
                    }
                }
#pragma unroll
                for (int q = 0; q < NR; ++q) mine[q] = next[q];
            }
#pragma unroll
            for (int q = 0; q < NR; ++q) {
                if (valid[q] && lane < k) {
                    const long long node = base + (long long)r[q] * k + lane;
                    const double confidence = (double)key_value(mine[q]) - lse[q];  // log c_i
                    const double v = parent_value[q] + confidence;
                    tok[node] = (int32_t)key_index(mine[q]);
                    par[node] = parent[q];
                    val[node] = v;
                    // the next frontier is ranked by value, or by confidence alone in the ablation
                    s_rank[r[q] * k + lane] = order_code_f64(by_confidence ? confidence : v);
                }
            }
        }
    };
    // The usual shape - at most 320 segment winners per row - takes a path written for the block that
    // runs it once per launch with none of its instructions in the cache: plain loops, no sorting
    // network.  Half a warp serves a row (the ten rows of a step on eight warps in one go): a lane holds
    // twenty of the row's keys; the k-th largest of the maxima of 32 groups of ten is a threshold that k keys reach; the keys
    // at or above it (a few dozen) go to the half-warp's list in shared memory and are ranked there by
    // counting.  all_ok turns false (and the general path redoes the step) when a list would overflow
    // (ties, rows of equal logits) or a row has fewer keys than children (tiny vocabularies).
    constexpr int kCompactBatch = 20, kHalfList = kWarpList / 2;
    bool compact_done = false;
    if (warp < kScanWarps && keys_per_row <= 16 * kCompactBatch) {
        const int hw = lane >> 4, hl = lane & 15;
        auto half_max_u64 = [](unsigned long long v) {
#pragma unroll
            for (int o = 8; o > 0; o >>= 1) {
                const unsigned long long other = __shfl_xor_sync(0xffffffffu, v, o);
                v = other > v ? other : v;
            }
            return v;
        };
        bool all_ok = true;
#pragma unroll 1
        for (int r0 = 0; r0 < n_s; r0 += 2 * kScanWarps) {
            const int r = r0 + warp * 2 + hw;
            const bool valid = r < n_s;
            const size_t p0 = ((size_t)b * n_s + (valid ? r : 0)) * chunks;
            unsigned long long cand[kCompactBatch];
#pragma unroll
            for (int t = 0; t < kCompactBatch; ++t)
                cand[t] = (valid && hl + 16 * t < keys_per_row) ? ws.keys[p0 * k + hl + 16 * t] : 0ull;
            // log-sum-exp of the row from the chunk partials, in double
            double mx = -INFINITY;
            if (valid)
                for (int c = hl; c < chunks; c += 16) mx = fmax(mx, ws.stats[p0 + c].x);
#pragma unroll
            for (int o = 8; o > 0; o >>= 1) mx = fmax(mx, __shfl_xor_sync(0xffffffffu, mx, o));
            double sum = 0.0;
            if (valid)
                for (int c = hl; c < chunks; c += 16) {
                    const double2 st = ws.stats[p0 + c];
                    if (st.x > -INFINITY) sum += st.y * exp(st.x - mx);
                }
#pragma unroll
            for (int o = 8; o > 0; o >>= 1) sum += __shfl_xor_sync(0xffffffffu, sum, o);
            if (valid && !(mx > -INFINITY)) status |= EAGLE2_STATUS_NONFINITE_LOGIT;
            const double lse = mx + log(sum);
            int parent = (s && valid) ? s_parent[r] : -1;
            const double parent_value = (s && valid) ? s_pvalue[r] : 0.0;
            if (parent < -1) {
                status |= EAGLE2_STATUS_BAD_TREE;
                parent = (int)(s >= 2 ? (long long)k + (long long)(s - 2) * k * k : 0);
            }
            // threshold: the k-th largest of 32 group maxima, two groups of ten keys per lane (0 when fewer
            // than k groups hold keys); with 32 groups a dozen keys reach it, with 16 several dozen would
            unsigned long long best_a = 0ull, best_b = 0ull;
#pragma unroll
            for (int t = 0; t < kCompactBatch / 2; ++t) {
                best_a = cand[t] > best_a ? cand[t] : best_a;
                best_b = cand[kCompactBatch / 2 + t] > best_b ? cand[kCompactBatch / 2 + t] : best_b;
            }
            int above_a = 0, above_b = 0;
#pragma unroll 4
            for (int l = 0; l < 16; ++l) {
                const unsigned long long oa = __shfl_sync(0xffffffffu, best_a, l, 16);
                const unsigned long long ob = __shfl_sync(0xffffffffu, best_b, l, 16);
                above_a += (oa > best_a) + (ob > best_a);
                above_b += (oa > best_b) + (ob > best_b);
            }
            unsigned long long pick = above_a == k - 1 ? best_a : 0ull;
            if (above_b == k - 1 && best_b > pick) pick = best_b;
            const unsigned long long thr = half_max_u64(pick);
            // the keys that reach it, packed into the half-warp's list
            unsigned long long* list = s_list[warp] + hw * kHalfList;
            int n_c = 0;
#pragma unroll
            for (int t = 0; t < kCompactBatch; ++t) {
                const bool in = cand[t] != 0ull && cand[t] >= thr;
                const unsigned mask = (__ballot_sync(0xffffffffu, in) >> (hw * 16)) & 0xffffu;
                const int pos = n_c + __popc(mask & ((1u << hl) - 1u));
                if (in && pos < kHalfList) list[pos] = cand[t];
                n_c += __popc(mask);
            }
            __syncwarp();
            if (valid && (n_c > kHalfList || n_c < k)) all_ok = false;
            const int n_l = min(n_c, kHalfList);
            // rank by counting (keys differ): the ranks below k are the row's children, best first
#pragma unroll 1
            for (int i = hl; i < n_l; i += 16) {
                const unsigned long long mine = list[i];
                int rank = 0;
#pragma unroll 4
                for (int j = 0; j < n_l; ++j) rank += list[j] > mine;
                if (valid && rank < k) {
                    const long long node = base + (long long)r * k + rank;
                    const double confidence = (double)key_value(mine) - lse;  // log c_i
                    const double v = parent_value + confidence;
                    tok[node] = (int32_t)key_index(mine);
                    par[node] = parent;
                    val[node] = v;
                    s_rank[r * k + rank] = order_code_f64(by_confidence ? confidence : v);
                }
            }
            __syncwarp();
        }
        compact_done = __all_sync(0xffffffffu, all_ok);
    }
    // every warp agrees on whether the general path has to redo the step (rare: ties, tiny vocabularies)
    compact_done = __syncthreads_and(compact_done || warp >= kScanWarps) && keys_per_row <= 16 * kCompactBatch;
    if (!compact_done && warp < kScanWarps) {
        using std::integral_constant;
        if (n_s > kScanWarps && n_s <= 2 * kScanWarps && keys_per_row <= 32 * 10)
            merge_rows(integral_constant<int, 2>{}, integral_constant<int, 10>{});
        else
            merge_rows(integral_constant<int, 1>{}, integral_constant<int, 16>{});
    }
    __syncthreads();  // all rows merged (the old frontier was read when the kernel started)

    // next frontier: rank the new candidates by (value desc, index asc); ranks < k are kept
    for (int i = threadIdx.x; i < n_new && threadIdx.x < kScanThreads; i += kScanThreads) {
        const unsigned long long ci = s_rank[i];
        int rank = 0;
#pragma unroll 8
        for (int j = 0; j < n_new; ++j) {
            const unsigned long long cj = s_rank[j];
            rank += (cj > ci) || (cj == ci && j < i);
        }
        if (rank < k) fr[rank] = (int32_t)(base + i);
    }
    if (status && lane == 0) raise_status(d_status, status);
}

// Phase 1 has no block-wide barrier inside the streaming loop.  Every streaming warp keeps, per
// lane, a running (max, sum of exponentials) of the elements it has seen, and filters its elements
// against a bar: a value that the k-th best element of the segment so far is known to reach, so that
// an element below it cannot be among the segment's k best.  The bar is shared by the block (a value
// code in shared memory that only rises).  Until there is one, a warp uses the k-th largest of its
// lanes' maxima of the tile at hand (at least k elements reach it).
//
// STREAM = false (one tile per block, the latency case): each warp lists its candidates (at most 64;
// more - ordered input, ties - are ranked exactly by k selection rounds), reduces them to its k best,
// and the block ranks the warps' 8k keys by counting.
// STREAM = true (several tiles per block): a ninth warp, the selector, owns the segment's k best.
// The streaming warps push candidates into a ring in shared memory; the selector takes them 32 at a
// time, merges them into its sorted 32 best (one key per lane) and raises the bar to the k-th.  How
// far behind the selector is changes only how many needless candidates are pushed, never the result.
//
// With 16-byte aligned rows each lane copies its own four float4 of a tile asynchronously into the
// warp's ring in shared memory, two tiles ahead, and reads back only what it copied itself; other
// rows are prefetched one tile ahead into registers.
template <bool VEC, bool STREAM>
__global__ void __launch_bounds__(STREAM ? kScanThreads + 32 : kScanThreads, 3)
expand_kernel(const float* __restrict__ draft_logits, long long batch_stride, int V, int k, int D,
              int s, int n_s, int chunks, int tpb, int by_confidence, int32_t* __restrict__ tree_token,
              int32_t* __restrict__ tree_parent, double* __restrict__ tree_value,
              int32_t* __restrict__ frontier, ExpandWs ws, long long wait_limit, int32_t* d_status) {
    constexpr int VPT = 4, NE = 16;
    constexpr float kLog2e = 1.4426950408889634f;
    extern __shared__ __align__(16) float s_ring[];  // [kScanWarps][kDepth][512] (vector path)
    __shared__ unsigned long long s_list[kScanWarps][kWarpList];  // !STREAM: the warps' candidate lists
    __shared__ unsigned long long s_queue[kQueue];  // STREAM: keys on their way to the selector (0: empty);
                                                     // otherwise: the block's surviving candidates at the end
    __shared__ int s_count[kScanWarps];
    __shared__ int s_tail, s_head, s_done;  // STREAM: slots reserved / consumed, streaming warps finished
                                            // (otherwise s_tail counts the surviving candidates)
    __shared__ uint32_t s_bar_code;         // the bar as a value code (0: none yet)
    __shared__ float s_wmax[kScanWarps], s_wsum[kScanWarps];
    __shared__ int s_flag;
    __shared__ unsigned long long s_rank[EAGLE2_MAX_K * EAGLE2_MAX_K];  // the new candidates' value codes

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    if (threadIdx.x == 0) s_bar_code = 0u, s_tail = 0, s_head = 0, s_done = 0;
    if (lane == 0 && warp < kScanWarps) s_count[warp] = 0;
    if (STREAM && threadIdx.x < kQueue) s_queue[threadIdx.x] = 0ull;
    __syncthreads();  // the only block-wide barrier before the segment's end
    // (which row and tiles this block serves is worked out before it waits for the preceding kernel)
    const int chunk = blockIdx.x % chunks;
    const int row = (blockIdx.x / chunks) % n_s;
    const int b = blockIdx.x / (chunks * n_s);
    const float* zrow = draft_logits + (long long)b * batch_stride + (long long)row * V;
    const int tiles = (V + kTileTokens - 1) / kTileTokens;
    const int t0 = chunk * tpb, t1 = min(tiles, t0 + tpb);
    const size_t part = ((size_t)b * n_s + row) * chunks + chunk;
    const long long N = nodes_of(k, D);
    int my_parent = -1;
    double my_parent_value = 0.0;
    int timed_out = 0;

    if (!STREAM || warp < kScanWarps) {
    // ===== streaming warps ==============================================================================
    // Vector path: float4 i of this lane sits 4096 bytes * i past the lane's first one in global
    // memory and 512 bytes * i past it in the warp's ring slot.
    const float* ring_lane = s_ring + (size_t)warp * kDepth * (32 * NE) + lane * 4;
    const uint32_t ring_addr = smem_addr(ring_lane);
    const float* src_next = zrow + (size_t)t0 * kTileTokens + threadIdx.x * 4;  // of the next tile to request
    int t_issue = t0, slot_issue = 0;
    auto issue_next = [&]() {  // requests one more tile (nothing once the segment is exhausted); one group each
        if (t_issue < t1) {
            const uint32_t dst = ring_addr + (uint32_t)slot_issue * (32 * NE * 4);
            if ((t_issue + 1) * kTileTokens <= V) {
#pragma unroll
                for (int i = 0; i < VPT; ++i) async_copy16(dst + i * 512, src_next + i * (kScanThreads * 4));
            } else {  // pieces past the row's end are skipped
#pragma unroll
                for (int i = 0; i < VPT; ++i)
                    if (scan_elem_index<VPT, true>(t_issue, 4 * i) < V) async_copy16(dst + i * 512, src_next + i * (kScanThreads * 4));
            }
        }
        async_commit();
        ++t_issue;
        src_next += kTileTokens;
        slot_issue = slot_issue == kDepth - 1 ? 0 : slot_issue + 1;
    };
    float cur[NE], nxt[NE];
    chain_wait();
    chain_release();
    if (VEC) {
        issue_next();
        issue_next();
    } else {
        scan_load<VPT, false>(zrow, V, t0, cur);
    }
    // The block that arrives last merges every row and then needs the rows' parents and their
    // values; whichever block that will be, the two dependent loads are already under way.
    if (s && threadIdx.x < n_s) {
        my_parent = frontier[(long long)b * k + threadIdx.x];
        const long long prev_base = s >= 2 ? (long long)k + (long long)(s - 2) * k * k : 0;
        const long long prev_count = s >= 2 ? (long long)k * k : k;
        if (my_parent < prev_base || my_parent >= prev_base + prev_count) my_parent = -2;  // reported by the merger
        else my_parent_value = tree_value[(long long)b * N + my_parent];
    }

    unsigned long long* list = s_list[warp];
    int n = 0;                          // !STREAM: keys in the list (warp-uniform; s_count[warp] mirrors it)
    float m_t = -INFINITY, s_t = 0.f;  // this thread's running maximum and sum of exp(x - m_t)

    auto push = [&](int pos, unsigned long long key) {  // STREAM: entry pos of the ring
        if (pos - *reinterpret_cast<volatile int*>(&s_head) >= kQueue) {  // the slot still holds entry pos - kQueue
            const long long w0 = clock64();
            while (pos - *reinterpret_cast<volatile int*>(&s_head) >= kQueue) {
                if (clock64() - w0 > wait_limit) {
                    timed_out = 1;
                    return;
                }
            }
        }
        *reinterpret_cast<volatile unsigned long long*>(&s_queue[pos & (kQueue - 1)]) = key;
    };
    auto consume = [&](int t, auto ragged_tag) {
        constexpr bool RAGGED = decltype(ragged_tag)::value;  // the tile reaches past the row's end
        float gm[VPT];  // maxima of the four float4
#pragma unroll
        for (int i = 0; i < VPT; ++i)
            gm[i] = fmaxf(fmaxf(cur[4 * i], cur[4 * i + 1]), fmaxf(cur[4 * i + 2], cur[4 * i + 3]));
        const float tm = fmaxf(fmaxf(gm[0], gm[1]), fmaxf(gm[2], gm[3]));
        if (tm > m_t) {
            s_t *= fast_ex2((m_t - tm) * kLog2e);  // 0 when nothing was summed yet
            m_t = tm;
        }
        if (m_t > -INFINITY) {
            // packed pairs: two elements per multiply-add and per addition, four chains of additions
            const float2 scale2 = make_float2(kLog2e, kLog2e), neg2 = make_float2(-m_t * kLog2e, -m_t * kLog2e);
            float2 acc_a = make_float2(0.f, 0.f), acc_b = make_float2(0.f, 0.f);
#pragma unroll
            for (int j = 0; j < NE; j += 4) {
                float2 a = __ffma2_rn(make_float2(cur[j], cur[j + 1]), scale2, neg2);
                float2 c2 = __ffma2_rn(make_float2(cur[j + 2], cur[j + 3]), scale2, neg2);
                a.x = fast_ex2(a.x), a.y = fast_ex2(a.y), c2.x = fast_ex2(c2.x), c2.y = fast_ex2(c2.y);
                acc_a = __fadd2_rn(acc_a, a);
                acc_b = __fadd2_rn(acc_b, c2);
            }
            s_t += (acc_a.x + acc_a.y) + (acc_b.x + acc_b.y);
        }
        const uint32_t block_code = *reinterpret_cast<volatile uint32_t*>(&s_bar_code);
        float thr = block_code ? order_decode(block_code) : -INFINITY;
        if (thr == -INFINITY) {
            thr = __shfl_sync(0xffffffffu, warp_sort_desc_f32(tm), k - 1);
            // k lanes hold an element that reaches it: a valid bar (if it is not -inf itself)
            if (lane == 0 && thr > -INFINITY) atomicMax(&s_bar_code, order_code(thr));
        }
        if (STREAM && t == t0) {
            // Once per block the streaming warps wait for each other's first bars: the largest of them
            // lets a handful of the first tile's elements through instead of a dozen per warp, which
            // is what the selector would otherwise spend the block's first microseconds on.
            asm volatile("bar.sync 1, %0;" ::"n"(kScanThreads) : "memory");
            const uint32_t code = *reinterpret_cast<volatile uint32_t*>(&s_bar_code);
            if (code) thr = fmaxf(thr, order_decode(code));
        }
        if (!__any_sync(0xffffffffu, tm >= thr)) return;
        uint32_t pmask = 0;  // this lane's candidates
        if (tm >= thr) {
#pragma unroll
            for (int j = 0; j < NE; ++j)
                if (cur[j] >= thr && (!RAGGED || scan_elem_index<VPT, VEC>(t, j) < V)) pmask |= 1u << j;
        }
        const int c = __popc(pmask);
        if constexpr (STREAM) {
            if (__any_sync(0xffffffffu, c >= NE / 2)) {
                // ordered input or ties: the tile's k best of this warp, ranked exactly, are all it can
                // contribute
                unsigned long long mine[NE];
#pragma unroll
                for (int j = 0; j < NE; ++j)
                    mine[j] = (pmask >> j) & 1u ? make_key(cur[j], (uint32_t)scan_elem_index<VPT, VEC>(t, j)) : 0ull;
                __syncwarp();
                warp_select<NE>(mine, k, list);
                __syncwarp();
                const unsigned long long key = lane < k ? list[lane] : 0ull;
                const uint32_t have = __ballot_sync(0xffffffffu, key != 0ull);
                int pos = 0;
                if (lane == 0) pos = atomicAdd(&s_tail, __popc(have));
                pos = __shfl_sync(0xffffffffu, pos, 0);
                if (key) push(pos + __popc(have & ((1u << lane) - 1u)), key);
                __syncwarp();
            } else if (c) {
                int pos = atomicAdd(&s_tail, c);
#pragma unroll
                for (int j = 0; j < NE; ++j)
                    if ((pmask >> j) & 1u) push(pos++, make_key(cur[j], (uint32_t)scan_elem_index<VPT, VEC>(t, j)));
            }
        } else {
            if (c) {
                int pos = atomicAdd(&s_count[warp], c);
                if (pos + c <= kWarpList) {  // else the count says "overflow" and the exact path takes over
#pragma unroll
                    for (int j = 0; j < NE; ++j)
                        if ((pmask >> j) & 1u) list[pos++] = make_key(cur[j], (uint32_t)scan_elem_index<VPT, VEC>(t, j));
                }
            }
            __syncwarp();
            const int n_new = *reinterpret_cast<volatile int*>(&s_count[warp]);
            if (n_new <= kWarpList) {
                n = n_new;
            } else {
                // exact: the k best of (the list as it was | this tile's candidates), lower index first
                // among equal values
                unsigned long long mine[NE + 2];
#pragma unroll
                for (int j = 0; j < NE; ++j)
                    mine[j] = (pmask >> j) & 1u ? make_key(cur[j], (uint32_t)scan_elem_index<VPT, VEC>(t, j)) : 0ull;
                mine[NE] = lane < n ? list[lane] : 0ull;
                mine[NE + 1] = lane + 32 < n ? list[lane + 32] : 0ull;
                __syncwarp();
                warp_select<NE + 2>(mine, k, list);
                __syncwarp();
                const unsigned long long kth = list[k - 1];
                n = __popc(__ballot_sync(0xffffffffu, lane < k && list[lane] != 0ull));  // the keys that exist
                if (lane == 0) {
                    s_count[warp] = n;
                    if (kth) atomicMax(&s_bar_code, (uint32_t)(kth >> 32));
                }
                __syncwarp();
            }
        }
    };

    int slot_read = 0;
    for (int t = t0; t < t1; ++t) {
        const bool ragged = (t + 1) * kTileTokens > V;
        if (VEC) {
            issue_next();
            async_wait<2>();  // tile t has landed; t+1 and t+2 may still be in flight
            const float4* slot = reinterpret_cast<const float4*>(ring_lane + slot_read * (32 * NE));
            slot_read = slot_read == kDepth - 1 ? 0 : slot_read + 1;
            if (!ragged) {
#pragma unroll
                for (int i = 0; i < VPT; ++i) {
                    const float4 v = slot[i * 32];
                    cur[4 * i + 0] = v.x, cur[4 * i + 1] = v.y, cur[4 * i + 2] = v.z, cur[4 * i + 3] = v.w;
                }
            } else {
#pragma unroll
                for (int i = 0; i < VPT; ++i) {
                    float4 v = make_float4(-INFINITY, -INFINITY, -INFINITY, -INFINITY);
                    if (scan_elem_index<VPT, true>(t, 4 * i) < V) v = slot[i * 32];
                    cur[4 * i + 0] = v.x, cur[4 * i + 1] = v.y, cur[4 * i + 2] = v.z, cur[4 * i + 3] = v.w;
                }
            }
        } else if (t + 1 < t1) {
            scan_load<VPT, false>(zrow, V, t + 1, nxt);
        }
        if (ragged) consume(t, std::true_type{});
        else consume(t, std::false_type{});
        if (!VEC) {
#pragma unroll
            for (int j = 0; j < NE; ++j) cur[j] = nxt[j];
        }
    }

    // ---- the warp's share of the segment's partial ---------------------------------------------------
    const float wmax = warp_max_f32(m_t);
    float scaled = m_t > -INFINITY ? s_t * fast_ex2((m_t - wmax) * kLog2e) : 0.f;
    scaled = warp_sum_f32(scaled);
    if (lane == 0) s_wmax[warp] = wmax, s_wsum[warp] = scaled;
    const int bad = !(scaled == scaled) || wmax == INFINITY;  // a NaN or +Inf logit poisons the sum / the max
    if (bad) raise_status(d_status, EAGLE2_STATUS_NONFINITE_LOGIT);
    if constexpr (STREAM) {
        __threadfence_block();  // the pushes and the statistics come before the count below
        __syncwarp();
        if (lane == 0) atomicAdd(&s_done, 1);
    } else {
        if (lane == 0) s_count[warp] = n;
    }
    } else {
    // ===== selector warp (STREAM) ==========================================================================
    chain_wait();
    chain_release();
    unsigned long long top = 0ull;  // the segment's best keys so far, descending over the lanes
    int head = 0;
    const long long w0 = clock64();
    for (;;) {
        const int done = *reinterpret_cast<volatile int*>(&s_done);  // read before the tail
        const int tail = *reinterpret_cast<volatile int*>(&s_tail);
        const int take = min(tail - head, 32);
        if (take <= 0) {
            if (done == kScanWarps) break;  // every reservation was made before its warp counted itself
            if (clock64() - w0 > 4 * wait_limit) {
                timed_out = 1;
                break;
            }
            __nanosleep(32);
            continue;
        }
        unsigned long long key = 0ull;
        if (lane < take) {
            volatile unsigned long long* slot = &s_queue[(head + lane) & (kQueue - 1)];
            const long long w1 = clock64();
            while ((key = *slot) == 0ull) {  // reserved, not yet written
                if (clock64() - w1 > wait_limit) {
                    timed_out = 1;
                    break;
                }
            }
            *slot = 0ull;
        }
        __threadfence_block();  // the slots are empty before the head says so
        __syncwarp();
        head += take;
        if (lane == 0) *reinterpret_cast<volatile int*>(&s_head) = head;
        // keys pushed under an older bar may already be beaten by the current k-th: nothing to merge
        const unsigned long long kth_now = __shfl_sync(0xffffffffu, top, k - 1);
        if (key <= kth_now) key = 0ull;
        if (!__any_sync(0xffffffffu, key != 0ull)) continue;
        const uint32_t fresh = __ballot_sync(0xffffffffu, key != 0ull);
        if (__popc(fresh) <= 6) {
            // a few keys: each is inserted at its place among the sorted 32 (the last one drops out)
            for (uint32_t left = fresh; left; left &= left - 1) {
                const unsigned long long x = __shfl_sync(0xffffffffu, key, __ffs(left) - 1);
                const int at = __popc(__ballot_sync(0xffffffffu, top > x));  // keys that stay ahead of x
                const unsigned long long up = __shfl_up_sync(0xffffffffu, top, 1);
                top = lane < at ? top : (lane == at ? x : up);
            }
        } else {
            // the 32 best of (top | the new keys): sort the new keys, pair the two sorted runs end to
            // end, keep the larger of each pair, sort the bitonic result
            key = warp_sort_desc_u64(key);
            const unsigned long long rev = __shfl_sync(0xffffffffu, key, 31 - lane);
            top = warp_bitonic_merge_desc(top > rev ? top : rev);
        }
        const unsigned long long kth = __shfl_sync(0xffffffffu, top, k - 1);
        if (lane == 0 && kth) atomicMax(&s_bar_code, (uint32_t)(kth >> 32));
    }
    if (lane < k) ws.keys[part * k + lane] = top;  // zeros where fewer than k keys exist
    // the warps' statistics were written before they counted themselves done
    const float pm = lane < kScanWarps ? *reinterpret_cast<volatile float*>(&s_wmax[lane]) : -INFINITY;
    const float cmax = warp_max_f32(pm);
    float term = 0.f;
    if (lane < kScanWarps && pm > -INFINITY)
        term = *reinterpret_cast<volatile float*>(&s_wsum[lane]) * fast_ex2((pm - cmax) * kLog2e);
    const float csum = warp_sum_f32(term);
    if (lane == 0) ws.stats[part] = make_double2((double)cmax, (double)csum);
    }
    if (timed_out) raise_status(d_status, EAGLE2_STATUS_TIMEOUT);

    if constexpr (!STREAM) {
        __syncthreads();
        // The block's k-th best reaches the largest of the warps' bars, so only the listed candidates
        // at or above it can be among the block's k best: usually a couple of dozen.  They are
        // gathered and every one is ranked by counting the ones above it (keys differ, so ranks do);
        // the ranks below k are the winners' places.
        const uint32_t bar_code = s_bar_code;
        const int n_w = s_count[warp];
#pragma unroll
        for (int u = 0; u < kWarpList / 32; ++u) {
            const unsigned long long key = lane + 32 * u < n_w ? s_list[warp][lane + 32 * u] : 0ull;
            if (key && (uint32_t)(key >> 32) >= bar_code) {
                const int pos = atomicAdd(&s_tail, 1);
                if (pos < kQueue) s_queue[pos] = key;
            }
        }
        __syncthreads();
        const int n_final = s_tail;
        if (n_final <= kQueue) {
            const unsigned long long mine = (int)threadIdx.x < n_final ? s_queue[threadIdx.x] : 0ull;
            if (mine) {
                int rank = 0;
#pragma unroll 8
                for (int j = 0; j < n_final; ++j) rank += s_queue[j] > mine;
                if (rank < k) ws.keys[part * k + rank] = mine;
            }
            if ((int)threadIdx.x >= n_final && (int)threadIdx.x < k) ws.keys[part * k + threadIdx.x] = 0ull;
        } else {
            // no useful bar (ties, rows of -inf): every warp reduces its list to its k best, then the
            // 8k keys are ranked in the same way
            unsigned long long* list = s_list[warp];
            if (n_w > 32) {
                unsigned long long two[2] = {list[lane], lane + 32 < n_w ? list[lane + 32] : 0ull};
                __syncwarp();
                warp_select<2>(two, k, list);
            } else {
                const unsigned long long sorted = warp_sort_desc_u64(lane < n_w ? list[lane] : 0ull);
                __syncwarp();
                if (lane < k) list[lane] = sorted;  // zeros where fewer than k keys exist
            }
            __syncthreads();
            const int n_keys = kScanWarps * k;  // <= 256 = threads
            const unsigned long long mine = (int)threadIdx.x < n_keys ? s_list[threadIdx.x / k][threadIdx.x % k] : 0ull;
            int rank = 0;
            if (mine) {
                for (int w = 0; w < kScanWarps; ++w)
                    for (int r = 0; r < k; ++r) rank += s_list[w][r] > mine;
                if (rank < k) ws.keys[part * k + rank] = mine;
            }
            const int present = __syncthreads_count(mine != 0ull);
            if ((int)threadIdx.x >= present && (int)threadIdx.x < k) ws.keys[part * k + threadIdx.x] = 0ull;
        }
        if (warp == 0) {
            const float pm = lane < kScanWarps ? s_wmax[lane] : -INFINITY;
            const float cmax = warp_max_f32(pm);
            float term = 0.f;
            if (lane < kScanWarps && pm > -INFINITY) term = s_wsum[lane] * fast_ex2((pm - cmax) * kLog2e);
            const float csum = warp_sum_f32(term);
            if (lane == 0) ws.stats[part] = make_double2((double)cmax, (double)csum);
        }
    }

    // ---- the last block of this sequence merges: a warp per row -------------------------------
    if (!last_block_arrives(ws.counters + b, chunks * n_s, &s_flag)) return;

    expand_finish(b, V, k, D, s, n_s, chunks, by_confidence, my_parent, my_parent_value, tree_token, tree_parent, tree_value,
                  frontier, ws, s_list, s_rank, d_status);
}

// Merge-only launch: one block per sequence finishes a step whose per-row partials (statistics and k
// best keys per producer, in this file's workspace layout with `chunks` producers per row) were
// written by another kernel - the LM head that ranks its own logits.
__global__ void __launch_bounds__(kScanThreads)
expand_merge_kernel(int V, int k, int D, int s, int n_s, int chunks, int by_confidence, int32_t* __restrict__ tree_token,
                    int32_t* __restrict__ tree_parent, double* __restrict__ tree_value,
                    int32_t* __restrict__ frontier, ExpandWs ws, int32_t* d_status) {
    __shared__ unsigned long long s_list[kScanWarps][kWarpList];
    __shared__ unsigned long long s_rank[EAGLE2_MAX_K * EAGLE2_MAX_K];
    chain_wait();
    chain_release();
    const int b = blockIdx.x;
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
    expand_finish(b, V, k, D, s, n_s, chunks, by_confidence, my_parent, my_parent_value, tree_token, tree_parent, tree_value,
                  frontier, ws, s_list, s_rank, d_status);
}

// Row-merge launch: one block per row folds the row's `chunks` partials into a single one (the same
// statistics and k best keys a lone producer would have written).  With a partial per SM a row has
// a few thousand keys, and a step's rows are independent: merging them side by side, a block each,
// leaves the per-sequence launch above only k keys per row.  Keys of a row are distinct (a token is
// ranked by exactly one producer) except for the empty slots, which hold 0.
constexpr int kRowMergeMaxKeysPerThread = 16;
__global__ void __launch_bounds__(kScanThreads)
expand_row_merge_kernel(int slots, int split_row, int chunks_lo, int chunks_hi, int k,
                        const double2* __restrict__ stats_in, const unsigned long long* __restrict__ keys_in,
                        double2* __restrict__ stats_out, unsigned long long* __restrict__ keys_out) {
    __shared__ unsigned long long s_top[kScanWarps * EAGLE2_MAX_K];  // every warp's k largest thread maxima
    __shared__ unsigned long long s_cand[kScanThreads];
    __shared__ unsigned long long s_thr;
    __shared__ int s_n;
    chain_wait();
    chain_release();
    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    const size_t row = blockIdx.x;
    const int chunks = (int)row < split_row ? chunks_lo : chunks_hi;  // producers that wrote this row
    const int n = chunks * k;
    const unsigned long long* kin = keys_in + row * (size_t)slots * k;
    unsigned long long mine[kRowMergeMaxKeysPerThread];
    unsigned long long mx[1] = {0ull};
#pragma unroll
    for (int t = 0; t < kRowMergeMaxKeysPerThread; ++t) {
        const int i = tid + t * kScanThreads;
        mine[t] = i < n ? kin[i] : 0ull;
        mx[0] = mine[t] > mx[0] ? mine[t] : mx[0];
    }
    if (tid == 0) s_n = 0, s_thr = 0ull;
    // The k-th largest of the threads' maxima is reached by at least k keys, and only the k threads
    // whose maximum reaches it can hold such keys: at most k * keys-per-thread candidates.
    warp_sort_desc_u64_n<1>(mx);
    if (lane < k) s_top[warp * k + lane] = mx[0];
    __syncthreads();
    if (tid < kScanWarps * k) {
        const unsigned long long v = s_top[tid];
        int above = 0;
        for (int j = 0; j < kScanWarps * k; ++j) {
            const unsigned long long w = s_top[j];
            above += (w > v) || (w == v && j < tid);
        }
        if (above == k - 1) s_thr = v;  // 0 when the row has fewer than k keys: every key is kept
    }
    // the row's log-sum-exp statistics from its partials, in double (one warp)
    if (warp == kScanWarps - 1) {
        const double2* sin = stats_in + row * (size_t)slots;
        double m = -INFINITY;
        for (int c = lane; c < chunks; c += 32) m = fmax(m, sin[c].x);
        m = warp_max_f64(m);
        double sum = 0.0;
        for (int c = lane; c < chunks; c += 32) {
            const double2 st = sin[c];
            if (st.x > -INFINITY) sum += st.y * exp(st.x - m);
        }
        sum = warp_sum_f64(sum);
        if (lane == 0) stats_out[row] = make_double2(m, sum);
    }
    __syncthreads();
    const unsigned long long thr = s_thr;
#pragma unroll
    for (int t = 0; t < kRowMergeMaxKeysPerThread; ++t) {
        if (mine[t] != 0ull && mine[t] >= thr) {
            const int pos = atomicAdd(&s_n, 1);
            if (pos < kScanThreads) s_cand[pos] = mine[t];
        }
    }
    __syncthreads();
    const int nc = min(s_n, kScanThreads);
    if (tid < nc) {
        const unsigned long long v = s_cand[tid];
        int above = 0;
        for (int j = 0; j < nc; ++j) above += s_cand[j] > v;
        if (above < k) keys_out[row * k + above] = v;
    }
    if (tid >= nc && tid < k) keys_out[row * k + tid] = 0ull;
}

// For the kernels of other files that write such partials: where they go in a workspace, how much of
// it they need, and the launch that finishes the step from them.
size_t expand_partials_bytes(int B, int n_s, int chunks, int k) { return expand_ws_layout(B, n_s, chunks, k, nullptr, nullptr); }
bool expand_partials_layout(int B, int n_s, int chunks, int k, void* ws, size_t ws_bytes, double2** stats,
                            unsigned long long** keys) {
    ExpandWs w;
    if (expand_ws_layout(B, n_s, chunks, k, ws, &w) > ws_bytes) return false;
    *stats = w.stats, *keys = w.keys;
    return true;
}
int launch_expand_merge(int B, int V, int k, int D, int s, int chunks, int32_t* tree_token, int32_t* tree_parent,
                        double* tree_value, int32_t* frontier, void* ws, int32_t* d_status, cudaStream_t stream) {
    const int n_s = s ? k : 1;
    ExpandWs w;
    expand_ws_layout(B, n_s, chunks, k, ws, &w);
    return launch_chained(expand_merge_kernel, dim3((unsigned)B), dim3(kScanThreads), 0, stream, 1, V, k, D, s, n_s, chunks,
                          0, tree_token, tree_parent, tree_value, frontier, w, d_status);
}

// Folds every row's partials into one per row, written in the same layout with one producer per row
// into `ws_rows`.  `ws` holds `slots` partial places per row, of which the first chunks_lo are filled
// for the rows below split_row and the first chunks_hi for the others (passes over the rows may use
// different numbers of producers).  Refuses more keys per row than the row-merge block holds.
int launch_expand_row_merge(int B, int n_s, int slots, long long split_row, int chunks_lo, int chunks_hi, int k, void* ws,
                            void* ws_rows, cudaStream_t stream) {
    const int most = chunks_lo > chunks_hi ? chunks_lo : chunks_hi;
    if (most > slots || (long long)most * k > (long long)kRowMergeMaxKeysPerThread * kScanThreads ||
        (long long)k * ((most * k + kScanThreads - 1) / kScanThreads) > kScanThreads)
        return EAGLE2_ERR_SHAPE;
    ExpandWs in, out;
    expand_ws_layout(B, n_s, slots, k, ws, &in);
    expand_ws_layout(B, n_s, 1, k, ws_rows, &out);
    const long long rows = (long long)B * n_s;
    return launch_chained(expand_row_merge_kernel, dim3((unsigned)rows), dim3(kScanThreads), 0, stream, 1, slots,
                          (int)(split_row < rows ? split_row : rows), chunks_lo, chunks_hi, k, in.stats, in.keys, out.stats,
                          out.keys);
}

template <bool VEC, bool STREAM>
static int launch_expand_as(const float* draft_logits, long long batch_stride, int B, int V, int k, int D,
                            int s, int n_s, int by_confidence, const ExpandPlan& plan, int32_t* tree_token,
                            int32_t* tree_parent,
                            double* tree_value, int32_t* frontier, const ExpandWs& ws, int32_t* d_status,
                            cudaStream_t stream) {
    const long long blocks = (long long)B * n_s * plan.chunks;
    const size_t dyn = VEC ? sizeof(float) * (size_t)kScanWarps * kDepth * 512 : 0;
    // the vector path's ring and the static arrays together exceed 48 KB
    if (VEC && cudaFuncSetAttribute(expand_kernel<VEC, STREAM>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                    (int)dyn) != cudaSuccess) {
        cudaGetLastError();
        return EAGLE2_ERR_CUDA;
    }
    return launch_chained(expand_kernel<VEC, STREAM>, dim3((unsigned)blocks),
                          dim3(STREAM ? kScanThreads + 32 : kScanThreads), dyn, stream, 1, draft_logits, batch_stride, V,
                          k, D, s, n_s, plan.chunks, plan.tpb, by_confidence, tree_token, tree_parent, tree_value,
                          frontier, ws, wait_limit_cycles(), d_status);
}

// Blocks that stream several tiles get the selector warp; one-tile blocks rank within the block.
template <bool VEC>
static int launch_expand(const float* draft_logits, long long batch_stride, int B, int V, int k, int D,
                         int s, int n_s, int by_confidence, const ExpandPlan& plan, int32_t* tree_token,
                         int32_t* tree_parent, double* tree_value, int32_t* frontier, const ExpandWs& ws,
                         int32_t* d_status, cudaStream_t stream) {
    return plan.tpb > 1 ? launch_expand_as<VEC, true>(draft_logits, batch_stride, B, V, k, D, s, n_s, by_confidence,
                                                      plan, tree_token, tree_parent, tree_value, frontier, ws,
                                                      d_status, stream)
                        : launch_expand_as<VEC, false>(draft_logits, batch_stride, B, V, k, D, s, n_s, by_confidence,
                                                       plan, tree_token, tree_parent, tree_value, frontier, ws,
                                                       d_status, stream);
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

// Expansion with a caller workspace; by_confidence selects the ablation's ranking score.
static int expand_with_workspace(const float* draft_logits, long long batch_stride, int B, int V, int k,
                                 int D, int s, int by_confidence, int32_t* tree_token,
                                 int32_t* tree_parent, double* tree_value, int32_t* frontier, void* ws,
                                 size_t ws_bytes, int32_t* d_status, eagle2_stream_t stream) {
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
    return vec ? launch_expand<true>(draft_logits, batch_stride, B, V, k, D, s, n_s, by_confidence, plan, tree_token,
                                     tree_parent, tree_value, frontier, w, d_status, st)
               : launch_expand<false>(draft_logits, batch_stride, B, V, k, D, s, n_s, by_confidence, plan, tree_token,
                                      tree_parent, tree_value, frontier, w, d_status, st);
}

extern "C" int eagle2_expand(const float* draft_logits, long long batch_stride, int B, int V, int k,
                             int D, int s, int32_t* tree_token, int32_t* tree_parent,
                             double* tree_value, int32_t* frontier, void* ws, size_t ws_bytes,
                             int32_t* d_status, eagle2_stream_t stream) {
    return expand_with_workspace(draft_logits, batch_stride, B, V, k, D, s, 0, tree_token, tree_parent, tree_value,
                                 frontier, ws, ws_bytes, d_status, stream);
}

extern "C" int eagle2_expand_variant(const float* draft_logits, long long batch_stride, int B, int V, int k,
                                     int D, int s, unsigned flags, int32_t* tree_token,
                                     int32_t* tree_parent, double* tree_value, int32_t* frontier, void* ws,
                                     size_t ws_bytes, int32_t* d_status, eagle2_stream_t stream) {
    if (flags & ~(unsigned)EAGLE2_EXPAND_BY_CONFIDENCE) return EAGLE2_ERR_SHAPE;
    return expand_with_workspace(draft_logits, batch_stride, B, V, k, D, s,
                                 (flags & EAGLE2_EXPAND_BY_CONFIDENCE) ? 1 : 0, tree_token, tree_parent,
                                 tree_value, frontier, ws, ws_bytes, d_status, stream);
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
    // the figure eagle2_workspace_bytes reports (the larger of the first step's and the later steps'
    // need) decides, so that every step of one tree is accepted or refused alike
    if (expand_workspace_bytes(B, V, k) > (size_t)EAGLE2_EXPAND_STATIC_BYTES) return EAGLE2_ERR_STATIC_LIMIT;
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
    return vec ? launch_expand<true>(draft_logits, batch_stride, B, V, k, D, s, n_s, 0, plan, tree_token, tree_parent,
                                     tree_value, frontier, w, d_status, st)
               : launch_expand<false>(draft_logits, batch_stride, B, V, k, D, s, n_s, 0, plan, tree_token,
                                      tree_parent, tree_value, frontier, w, d_status, st);
}
