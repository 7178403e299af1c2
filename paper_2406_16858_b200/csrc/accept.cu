// Step 4 of the hot path: acceptance over the draft tree (paper Section 2.1 rule, walked over the
// tree as described in Section 2.2).
//
// temperature == 0 (greedy): one launch.  Block (chunk, row, sequence) finds the arg-max of its
// chunk of a target row; the last block of the sequence merges the rows' arg-maxes and walks.
//
// temperature > 0 (multi-round speculative sampling over siblings): two launches.
//   chain kernel  One thread-block cluster per (sequence, expanded node).  The cluster keeps the
//     node's target and draft distributions in shared memory (each block a slice of the vocabulary,
//     read from HBM once) and runs the node's whole rejection chain over its selected children: the
//     acceptance threshold of every child under the hypothesis that all earlier siblings were
//     rejected.  This uses that the state after j rejections is a function of the ORIGINAL rows:
//       q_j = s_j * q_0 off the removed tokens,  s_j = 1 / (1 - sum_{i<j} q_0(x_i)),
//       p_j = max(p_0 - alpha(v) q_0, 0) / beta_j,  alpha_{j+1} = alpha_j + beta_j s_j,
//       beta_{j+1} = sum_v max(p_0 - alpha_{j+1}(v) q_0, 0),  a removed token keeping the alpha in
//       force when it was removed,
//     so a chain does not depend on the path taken and all nodes' chains run in parallel; each round
//     is one reduction over the on-chip slices, combined across the cluster through distributed
//     shared memory.
//   bonus kernel  Every block repeats the (tiny) walk with the thresholds and the caller's uniforms,
//     then the blocks of a sequence sum the weights of the distribution in force at the stopping node
//     chunk by chunk; the last block locates the inverse-CDF token.
#include <cooperative_groups.h>
#include <math.h>

#include "vocab_scan.cuh"

namespace cg = cooperative_groups;

namespace eagle2 {

// ------------------------------------------------------------------------------------------------
// shared conventions

// draft row that produced the children of a node, from the candidate index of any of its children
__device__ __forceinline__ int draft_row_of_child(int idx, int k) {
    if (idx < k) return 0;
    const int level = 2 + (idx - k) / (k * k);
    const int slot = ((idx - k) % (k * k)) / k;
    return 1 + (level - 2) * k + slot;
}

constexpr int kChainThreads = 512;
constexpr int kChainWarps = kChainThreads / kWarp;
constexpr int kMaxCluster = 8;
constexpr int kResidentSliceMax = 24576;  // floats per row slice kept in shared memory (2 rows)

struct ChainSlot {        // result of one node's rejection chain, read by the bonus kernel
    float gmax_p, gmax_q; // maxima of the scaled logits
    float c_p, c_q;       // 1 / sum exp(scaled - max)
    double alpha;         // alpha in force after the last round
    int n_children;
    int pad;
    double removed_alpha[EAGLE2_MAX_K];  // alpha frozen for child j's token (full-q mode)
    int removed[EAGLE2_MAX_K];           // point-mass mode: 1 if child j's token was taken out of p
};

struct AcceptWs {
    int* counters;              // [B]
    unsigned long long* keys;   // greedy: [B][m+1][chunks]
    double* thr;                // sampling: [B][m] acceptance thresholds
    ChainSlot* slots;           // sampling: [B][R]
    double2* bstats;            // sampling: [B][bchunks] (chunk max of scaled logits or 0, weight sum)
    int* blast;                 // sampling: [B][bchunks] last index with positive weight, or -1
};

static size_t accept_ws_layout(int B, int m, int R, int gchunks, int bchunks, void* base, AcceptWs* w) {
    size_t off = 0;
    char* p = static_cast<char*>(base);
#define EAGLE2_WS_FIELD(field, type, count)                          \
    if (w) w->field = reinterpret_cast<type*>(p + off);              \
    off += round_up(sizeof(type) * (size_t)(count), kWsAlign);
    if (w) w->counters = reinterpret_cast<int*>(p);
    off += counters_bytes(B);
    EAGLE2_WS_FIELD(keys, unsigned long long, (size_t)B * (m + 1) * gchunks)
    EAGLE2_WS_FIELD(thr, double, (size_t)B * m)
    EAGLE2_WS_FIELD(slots, ChainSlot, (size_t)B * R)
    EAGLE2_WS_FIELD(bstats, double2, (size_t)B * bchunks)
    EAGLE2_WS_FIELD(blast, int, (size_t)B * bchunks)
#undef EAGLE2_WS_FIELD
    return off;
}

static int greedy_vpt(int B, int m, int V) { return scan_pick_vpt((long long)B * (m + 1), V); }
static int bonus_vpt(int B, int V) { return scan_pick_vpt(B, V); }

size_t accept_workspace_bytes(int B, int V, int k, int D, int m) {
    const int R = 1 + (D - 1) * k;
    return accept_ws_layout(B, m, R, scan_chunks(V, greedy_vpt(B, m, V)), scan_chunks(V, bonus_vpt(B, V)),
                            nullptr, nullptr);
}

// ------------------------------------------------------------------------------------------------
// greedy

template <int VPT, bool VEC>
__global__ void __launch_bounds__(kScanThreads)
accept_greedy_kernel(const float* __restrict__ target_logits, long long t_stride,
                     const int32_t* __restrict__ sel_parent, const int32_t* __restrict__ sel_token,
                     const int32_t* __restrict__ n_sel, int V, int D, int m, int chunks,
                     int32_t* __restrict__ acc_len, int32_t* __restrict__ acc_path,
                     int32_t* __restrict__ bonus_token, AcceptWs ws, int32_t* d_status) {
    constexpr int NE = 4 * VPT;
    __shared__ unsigned long long s_keys[kScanWarps * EAGLE2_MAX_K];
    __shared__ int s_flag;
    __shared__ int s_arg[EAGLE2_MAX_M + 1];
    __shared__ int s_par[EAGLE2_MAX_M], s_tok[EAGLE2_MAX_M];

    const int chunk = blockIdx.x % chunks;
    const int row = (blockIdx.x / chunks) % (m + 1);
    const int b = blockIdx.x / (chunks * (m + 1));
    chain_wait();
    chain_release();
    const int ns = min(n_sel[b], m);
    const size_t part = ((size_t)b * (m + 1) + row) * chunks + chunk;

    if (row <= ns) {  // rows of padding nodes are never consulted
        const float* zrow = target_logits + (long long)b * t_stride + (long long)row * V;
        float x[NE];
        scan_load<VPT, VEC>(zrow, V, chunk, x);
        unsigned long long key[NE];
        int bad = 0;
#pragma unroll
        for (int j = 0; j < NE; ++j) {
            const int e = scan_elem_index<VPT, VEC>(chunk, j);
            bad |= (x[j] != x[j]);
            key[j] = e < V ? make_key(x[j], (uint32_t)e) : 0ull;
        }
        block_topk<NE>(key, 1, s_keys, ws.keys + part);
        if (bad) raise_status(d_status, EAGLE2_STATUS_NONFINITE_LOGIT);
    }
    if (!last_block_arrives(ws.counters + b, chunks * (m + 1), &s_flag)) return;

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    for (int r = warp; r <= ns; r += kScanWarps) {
        const size_t p0 = ((size_t)b * (m + 1) + r) * chunks;
        unsigned long long best = 0;
        for (int c = lane; c < chunks; c += 32) {
            const unsigned long long kk = ws.keys[p0 + c];
            best = kk > best ? kk : best;
        }
        best = warp_max_u64(best);
        if (lane == 0) s_arg[r] = (int)key_index(best);
    }
    for (int x = threadIdx.x; x < m; x += kScanThreads) {
        s_par[x] = sel_parent[(long long)b * m + x];
        s_tok[x] = sel_token[(long long)b * m + x];
    }
    __syncthreads();
    if (warp != 0) return;
    // the walk: follow the child whose token equals the arg-max of the current node's row
    int cur = -1, len = 0, bonus = 0;
    for (;;) {
        const int a = s_arg[cur + 1];
        bonus = a;
        int next = -1;
        for (int x0 = 0; x0 < ns && next < 0; x0 += 32) {
            const int x = x0 + lane;
            const bool hit = x < ns && x > cur && s_par[x] == cur && s_tok[x] == a;
            const unsigned mask = __ballot_sync(0xffffffffu, hit);
            if (mask) next = x0 + __ffs(mask) - 1;
        }
        if (next < 0 || len >= D) break;
        if (lane == 0) acc_path[(long long)b * D + len] = next;
        ++len;
        cur = next;
    }
    for (int j = len + lane; j < D; j += 32) acc_path[(long long)b * D + j] = -1;
    if (lane == 0) {
        acc_len[b] = len;
        bonus_token[b] = bonus;
    }
}

// ------------------------------------------------------------------------------------------------
// sampling: chain kernel

__device__ __forceinline__ double chain_block_sum(double v, double* s_red) {
    v = warp_sum_f64(v);
    __syncthreads();
    if ((threadIdx.x & 31) == 0) s_red[threadIdx.x >> 5] = v;
    __syncthreads();
    double r = 0.0;
#pragma unroll
    for (int w = 0; w < kChainWarps; ++w) r += s_red[w];
    return r;
}
// Two block-wide sums (or maxima) behind one pair of barriers.  s_red: 2 * kChainWarps entries.
__device__ __forceinline__ void chain_block_sum2(double& a, double& b, double* s_red) {
    a = warp_sum_f64(a), b = warp_sum_f64(b);
    __syncthreads();
    if ((threadIdx.x & 31) == 0) s_red[threadIdx.x >> 5] = a, s_red[kChainWarps + (threadIdx.x >> 5)] = b;
    __syncthreads();
    double ra = 0.0, rb = 0.0;
#pragma unroll
    for (int w = 0; w < kChainWarps; ++w) ra += s_red[w], rb += s_red[kChainWarps + w];
    a = ra, b = rb;
}
__device__ __forceinline__ void chain_block_max2(float& a, float& b, float* s_red) {
    a = warp_max_f32(a), b = warp_max_f32(b);
    __syncthreads();
    if ((threadIdx.x & 31) == 0) s_red[threadIdx.x >> 5] = a, s_red[kChainWarps + (threadIdx.x >> 5)] = b;
    __syncthreads();
    float ra = s_red[0], rb = s_red[kChainWarps];
#pragma unroll
    for (int w = 1; w < kChainWarps; ++w) ra = fmaxf(ra, s_red[w]), rb = fmaxf(rb, s_red[kChainWarps + w]);
    a = ra, b = rb;
}

// All-reduce of two doubles across the blocks of the cluster through distributed shared memory.
// Every thread passes the block's value; the result is the same in every block (fixed order).
template <bool IS_MAX>
__device__ __forceinline__ void cluster_allreduce2(cg::cluster_group& cluster, double& a, double& b,
                                                   double* s_xchg /*[2][kMaxCluster][2]*/, int& parity) {
    const unsigned cs = cluster.num_blocks(), me = cluster.block_rank();
    if (threadIdx.x < cs) {
        double* peer = cluster.map_shared_rank(s_xchg, threadIdx.x);
        peer[(parity * kMaxCluster + me) * 2 + 0] = a;
        peer[(parity * kMaxCluster + me) * 2 + 1] = b;
    }
    cluster.sync();
    double ra = s_xchg[(parity * kMaxCluster) * 2 + 0], rb = s_xchg[(parity * kMaxCluster) * 2 + 1];
    for (unsigned r = 1; r < cs; ++r) {
        const double xa = s_xchg[(parity * kMaxCluster + r) * 2 + 0];
        const double xb = s_xchg[(parity * kMaxCluster + r) * 2 + 1];
        ra = IS_MAX ? fmax(ra, xa) : ra + xa;
        rb = IS_MAX ? fmax(rb, xb) : rb + xb;
    }
    a = ra;
    b = rb;
    parity ^= 1;
}

// Probability of one token.  Explicit round-to-nearest operations (never contracted into an FMA)
// so that a token looked up on its own gets bit for bit the value its resident copy has.
__device__ __forceinline__ float scale_logit(float z, float inv_t) { return __fmul_rn(z, inv_t); }
// exp(zs - gmax) as 2^((zs - gmax) * log2 e) with the hardware's approximate 2^x (2 ulp); the
// difference and the product are separately rounded, so every caller gets the same bits for the same token
__device__ __forceinline__ float exp_scaled(float zs, float gmax) {
    float y;
    asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(__fmul_rn(__fsub_rn(zs, gmax), 1.4426950408889634f)));
    return y;
}
__device__ __forceinline__ float prob_of(float z, float inv_t, float gmax, float c) {
    return __fmul_rn(exp_scaled(scale_logit(z, inv_t), gmax), c);
}

template <bool RESIDENT, bool VEC>
__global__ void __launch_bounds__(kChainThreads)
accept_chain_kernel(const float* __restrict__ target_logits, long long t_stride,
                    const float* __restrict__ draft_logits_all, long long d_stride,
                    const int32_t* __restrict__ sel_index, const int32_t* __restrict__ sel_parent,
                    const int32_t* __restrict__ sel_token, const int32_t* __restrict__ n_sel,
                    const float* __restrict__ u_accept, int V, int k, int m, int R, int slice, float inv_t,
                    AcceptWs ws, int32_t* d_status) {
    cg::cluster_group cluster = cg::this_cluster();
    const int cs = (int)cluster.num_blocks(), me = (int)cluster.block_rank();
    const int b = blockIdx.x / cs;
    const int r = blockIdx.y;  // draft row = the expanded node whose children this cluster handles
    const int tid = threadIdx.x;
    chain_wait();
    chain_release();

    extern __shared__ __align__(16) float s_rows[];  // RESIDENT: p slice then q slice
    __shared__ double s_xchg[2 * kMaxCluster * 2];
    __shared__ double s_redd[2 * kChainWarps];
    __shared__ float s_redf[2 * kChainWarps];
    __shared__ int s_child[EAGLE2_MAX_K], s_ctok[EAGLE2_MAX_K];
    __shared__ float s_pf[EAGLE2_MAX_K], s_qf[EAGLE2_MAX_K], s_uc[EAGLE2_MAX_K];  // children's p, q, uniform
    __shared__ double s_frozen[EAGLE2_MAX_K];
    __shared__ int s_nchild, s_parent;

    // ---- which selected nodes are children produced by draft row r (same in every block) ------
    // every candidate is looked at by its own thread; ballots keep the ascending order
    __shared__ unsigned s_ballot[EAGLE2_MAX_M / 32];
    const int ns = min(n_sel[b], m);
    if (tid < EAGLE2_MAX_M) {
        const int x = tid;
        int tokx = 0, parx = -1;
        float ux = 0.f;
        bool match = false;
        if (x < ns) {
            const int idx = sel_index[(long long)b * m + x];
            match = idx >= 0 && draft_row_of_child(idx, k) == r;
            if (match) {
                tokx = sel_token[(long long)b * m + x];
                parx = sel_parent[(long long)b * m + x];
                ux = u_accept[(long long)b * m + x];
            }
        }
        const unsigned bal = __ballot_sync(0xffffffffu, match);
        if ((tid & 31) == 0) s_ballot[tid >> 5] = bal;
        asm volatile("bar.sync 1, %0;" ::"n"(EAGLE2_MAX_M) : "memory");  // the first four warps
        int before = __popc(bal & ((1u << (tid & 31)) - 1u)), total = 0;
        for (int w = 0; w < EAGLE2_MAX_M / 32; ++w) {
            const int c = __popc(s_ballot[w]);
            if (w < (tid >> 5)) before += c;
            total += c;
        }
        if (match && before < EAGLE2_MAX_K) {
            s_child[before] = x;
            s_ctok[before] = tokx;
            s_uc[before] = ux;
            if (before == 0) s_parent = parx;
        }
        if (tid == 0) s_nchild = min(total, EAGLE2_MAX_K);
    }
    __syncthreads();
    const int nc = s_nchild;
    ChainSlot* slot = ws.slots + (size_t)b * R + r;
    if (nc == 0) {  // nothing hangs below this row: the whole cluster leaves
        if (me == 0 && tid == 0) slot->n_children = 0;
        return;
    }
    cluster.sync();  // every block of the cluster runs before any remote shared-memory write
    const bool full_q = draft_logits_all != nullptr;
    const float* zp = target_logits + (long long)b * t_stride + (long long)(s_parent + 1) * V;
    const float* zq = full_q ? draft_logits_all + (long long)b * d_stride + (long long)r * V : nullptr;
    const int lo = me * slice, hi = min(V, lo + slice);
    const int n_local = max(hi - lo, 0);
    float* sp = s_rows;
    float* sq = s_rows + (RESIDENT ? slice : 0);
    int parity = 0, bad = 0;

    // ---- pass 1: scaled logits -> shared memory, maxima ---------------------------------------
    float mp = -INFINITY, mq = -INFINITY;
    if (VEC) {
        constexpr int kPre = 4;  // float4 per row requested before any is used
        for (int e0 = tid * 4; e0 < n_local; e0 += kChainThreads * 4 * kPre) {
            float4 a[kPre], c[kPre];
#pragma unroll
            for (int u = 0; u < kPre; ++u) {
                const int e = e0 + u * kChainThreads * 4;
                if (e < n_local) {
                    a[u] = __ldcs(reinterpret_cast<const float4*>(zp + lo + e));
                    if (full_q) c[u] = __ldcs(reinterpret_cast<const float4*>(zq + lo + e));
                }
            }
#pragma unroll
            for (int u = 0; u < kPre; ++u) {
                const int e = e0 + u * kChainThreads * 4;
                if (e >= n_local) continue;
                float4 x = a[u];
                x.x = scale_logit(x.x, inv_t), x.y = scale_logit(x.y, inv_t);
                x.z = scale_logit(x.z, inv_t), x.w = scale_logit(x.w, inv_t);
                bad |= !(x.x < INFINITY) | !(x.y < INFINITY) | !(x.z < INFINITY) | !(x.w < INFINITY);
                mp = fmaxf(fmaxf(mp, fmaxf(x.x, x.y)), fmaxf(x.z, x.w));
                if (RESIDENT) *reinterpret_cast<float4*>(sp + e) = x;
                if (full_q) {
                    float4 y = c[u];
                    y.x = scale_logit(y.x, inv_t), y.y = scale_logit(y.y, inv_t);
                    y.z = scale_logit(y.z, inv_t), y.w = scale_logit(y.w, inv_t);
                    bad |= !(y.x < INFINITY) | !(y.y < INFINITY) | !(y.z < INFINITY) | !(y.w < INFINITY);
                    mq = fmaxf(fmaxf(mq, fmaxf(y.x, y.y)), fmaxf(y.z, y.w));
                    if (RESIDENT) *reinterpret_cast<float4*>(sq + e) = y;
                }
            }
        }
    } else {
        for (int e = tid; e < n_local; e += kChainThreads) {
            const float a = scale_logit(__ldcs(zp + lo + e), inv_t);
            bad |= !(a < INFINITY);
            mp = fmaxf(mp, a);
            if (RESIDENT) sp[e] = a;
            if (full_q) {
                const float c = scale_logit(__ldcs(zq + lo + e), inv_t);
                bad |= !(c < INFINITY);
                mq = fmaxf(mq, c);
                if (RESIDENT) sq[e] = c;
            }
        }
    }
    chain_block_max2(mp, mq, s_redf);
    double gp = (double)mp, gq = (double)mq;
    cluster_allreduce2<true>(cluster, gp, gq, s_xchg, parity);
    const float gmax_p = (float)gp, gmax_q = (float)gq;
    if (!(gmax_p > -INFINITY) || (full_q && !(gmax_q > -INFINITY))) bad = 1;

    // ---- pass 2: exponentials (kept in place, unnormalised), sums -----------------------------------
    float tp = 0.f, tq = 0.f;
    if (RESIDENT && VEC) {
        for (int e = tid * 4; e < n_local; e += kChainThreads * 4) {
            float4 a = *reinterpret_cast<const float4*>(sp + e);
            a.x = exp_scaled(a.x, gmax_p), a.y = exp_scaled(a.y, gmax_p);
            a.z = exp_scaled(a.z, gmax_p), a.w = exp_scaled(a.w, gmax_p);
            tp += (a.x + a.y) + (a.z + a.w);
            *reinterpret_cast<float4*>(sp + e) = a;
            if (full_q) {
                float4 c = *reinterpret_cast<const float4*>(sq + e);
                c.x = exp_scaled(c.x, gmax_q), c.y = exp_scaled(c.y, gmax_q);
                c.z = exp_scaled(c.z, gmax_q), c.w = exp_scaled(c.w, gmax_q);
                tq += (c.x + c.y) + (c.z + c.w);
                *reinterpret_cast<float4*>(sq + e) = c;
            }
        }
    } else {
        for (int e = tid; e < n_local; e += kChainThreads) {
            const float a = exp_scaled(RESIDENT ? sp[e] : scale_logit(zp[lo + e], inv_t), gmax_p);
            tp += a;
            if (RESIDENT) sp[e] = a;
            if (full_q) {
                const float c = exp_scaled(RESIDENT ? sq[e] : scale_logit(zq[lo + e], inv_t), gmax_q);
                tq += c;
                if (RESIDENT) sq[e] = c;
            }
        }
    }
    double sum_p = (double)tp, sum_q = (double)tq;
    chain_block_sum2(sum_p, sum_q, s_redd);
    cluster_allreduce2<false>(cluster, sum_p, sum_q, s_xchg, parity);
    const float c_p = (float)(1.0 / sum_p), c_q = full_q ? (float)(1.0 / sum_q) : 0.f;
    // Residual mass sum_v max(p_0(v) - alpha q_0(v), 0) over this block's slice.  The resident copies
    // hold the unnormalised exponentials; p and q are formed on the fly with the same two roundings
    // as prob_of(), so a token looked up on its own has bit for bit the value used here.
    auto residual_mass = [&](float an) {
        float part = 0.f;
        if (RESIDENT && VEC) {
            for (int e = tid * 4; e < n_local; e += kChainThreads * 4) {
                const float4 a = *reinterpret_cast<const float4*>(sp + e);
                const float4 c = *reinterpret_cast<const float4*>(sq + e);
                part += fmaxf(fmaf(-an, __fmul_rn(c.x, c_q), __fmul_rn(a.x, c_p)), 0.f);
                part += fmaxf(fmaf(-an, __fmul_rn(c.y, c_q), __fmul_rn(a.y, c_p)), 0.f);
                part += fmaxf(fmaf(-an, __fmul_rn(c.z, c_q), __fmul_rn(a.z, c_p)), 0.f);
                part += fmaxf(fmaf(-an, __fmul_rn(c.w, c_q), __fmul_rn(a.w, c_p)), 0.f);
            }
        } else {
            for (int e = tid; e < n_local; e += kChainThreads) {
                const float pe = RESIDENT ? __fmul_rn(sp[e], c_p) : prob_of(zp[lo + e], inv_t, gmax_p, c_p);
                const float qe = RESIDENT ? __fmul_rn(sq[e], c_q) : prob_of(zq[lo + e], inv_t, gmax_q, c_q);
                part += fmaxf(fmaf(-an, qe, pe), 0.f);
            }
        }
        return part;
    };
    // the children's own probabilities, computed exactly like the resident values
    if (tid < nc) {
        const int t = s_ctok[tid];
        const bool ok = t >= 0 && t < V;
        if (!ok) bad = 1;
        s_pf[tid] = ok ? prob_of(zp[t], inv_t, gmax_p, c_p) : 0.f;
        s_qf[tid] = (ok && full_q) ? prob_of(zq[t], inv_t, gmax_q, c_q) : 0.f;
    }
    __syncthreads();
    if (bad) raise_status(d_status, EAGLE2_STATUS_NONFINITE_LOGIT);

    const bool writer = (me == 0 && tid == 0);
    double* thr = ws.thr + (size_t)b * m;

    if (!full_q) {
        // proposal = point mass on the candidate: accept with p_j(x), then take x out of p
        double removed_p = 0.0;
        for (int j = 0; j < nc; ++j) {
            const double px = (double)s_pf[j];
            const double rest = 1.0 - removed_p;
            const double pj = rest > 0.0 ? px / rest : 0.0;
            const double a = pj < 1.0 ? pj : 1.0;
            const bool take_out = (rest - px) > 0.0;  // zero residual mass: keep p as it is
            if (take_out) removed_p += px;
            if (writer) {
                thr[s_child[j]] = a;
                slot->removed[j] = take_out ? 1 : 0;
            }
        }
        if (writer) {
            slot->gmax_p = gmax_p, slot->gmax_q = 0.f, slot->c_p = c_p, slot->c_q = 0.f;
            slot->alpha = 0.0;
            slot->n_children = nc;
        }
        return;
    }

    // ---- the rejection chain over this node's children ------------------------------------------
    // (alpha, beta): the target in force is max(p_0 - alpha q_0, 0) / beta.  Every thread of every
    // block of the cluster carries the same scalars.
    double alpha = 0.0, beta = 1.0, removed_q = 0.0, s = 1.0;
    for (int j = 0; j < nc; ++j) {
        const double pf = (double)s_pf[j], qf = (double)s_qf[j];
        const double pj = fmax(pf - alpha * qf, 0.0) / beta;
        const double qj = s * qf;
        double a;
        if (qj > 0.0)
            a = pj / qj < 1.0 ? pj / qj : 1.0;
        else
            a = pj > 0.0 ? 1.0 : 0.0;
        if (writer) thr[s_child[j]] = a;
        // The walk takes the first child whose uniform is below its threshold and never looks at a
        // later sibling: the chain of this node ends here (same decision in every thread and block).
        if ((double)s_uc[j] < a) break;

        // residual after rejecting child j: alpha grows by beta * s for every token still in q
        const double alpha_new = alpha + beta * s;
        const float an = (float)alpha_new;
        if (j == nc - 1) {
            // nothing is tested after the last child: only alpha is needed (by the extra token's
            // law).  A rejection implies p < q at the rejected token, hence mass left elsewhere.
            alpha = alpha_new;
            if (tid == 0) s_frozen[j] = alpha;
            break;
        }
        double f_new, unused = 0.0;
        f_new = chain_block_sum((double)residual_mass(an), s_redd);
        cluster_allreduce2<false>(cluster, f_new, unused, s_xchg, parity);
        // tokens removed in earlier rounds keep the alpha in force when they were removed
        for (int i = 0; i < j; ++i) {
            const float pi = s_pf[i], qi = s_qf[i];
            f_new -= (double)fmaxf(fmaf(-an, qi, pi), 0.f);
            f_new += (double)fmaxf(fmaf(-(float)s_frozen[i], qi, pi), 0.f);
        }
        if (f_new > 0.0) {  // zero residual mass: the target stays as it is
            alpha = alpha_new;
            beta = f_new;
        }
        if (tid == 0) s_frozen[j] = alpha;
        removed_q += qf;
        const double rest = 1.0 - removed_q;
        s = rest > 0.0 ? 1.0 / rest : 0.0;
    }
    __syncthreads();
    if (writer) {
        slot->gmax_p = gmax_p, slot->gmax_q = gmax_q, slot->c_p = c_p, slot->c_q = c_q;
        slot->alpha = alpha;
        slot->n_children = nc;
        for (int j = 0; j < nc; ++j) slot->removed_alpha[j] = s_frozen[j];
    }
}

// ------------------------------------------------------------------------------------------------
// sampling: walk + extra token

struct WalkResult {
    int cur;        // flat node where the walk stopped (-1: root)
    int len;        // accepted draft tokens
    int slot_row;   // draft row of the stopping node's children if all were rejected, else -1
};

// Executed by warp 0 of a block; m <= 128.  s_par/s_thr/s_u hold the sequence's arrays.
__device__ __forceinline__ WalkResult walk_tree(const int* s_par, const double* s_thr, const float* s_u,
                                                const int32_t* sel_index_b, int ns, int k, int D,
                                                int32_t* path_out /* nullable, [D] */) {
    const int lane = threadIdx.x & 31;
    WalkResult w;
    w.cur = -1, w.len = 0, w.slot_row = -1;
    for (;;) {
        int first_child = -1, accepted = -1;
        for (int x0 = 0; x0 < ns; x0 += 32) {
            const int x = x0 + lane;
            const bool child = x < ns && x > w.cur && s_par[x] == w.cur;
            const bool take = child && ((double)s_u[x] < s_thr[x]);
            const unsigned cm = __ballot_sync(0xffffffffu, child);
            const unsigned tm = __ballot_sync(0xffffffffu, take);
            if (first_child < 0 && cm) first_child = x0 + __ffs(cm) - 1;
            if (accepted < 0 && tm) accepted = x0 + __ffs(tm) - 1;
        }
        if (first_child < 0 || w.len >= D) break;  // leaf (or depth budget): plain target
        if (accepted < 0) {                        // every child rejected: residual of this node
            w.slot_row = draft_row_of_child(sel_index_b[first_child], k);
            break;
        }
        if (path_out && lane == 0) path_out[w.len] = accepted;
        ++w.len;
        w.cur = accepted;
    }
    return w;
}

// weight of token e under the distribution in force at the stopping node
struct BonusLaw {
    const float* zp;
    const float* zq;
    float inv_t, gmax_p, gmax_q, c_p, c_q, alpha;
    int mode;  // 0: plain softmax (relative to a chunk maximum), 1: full-q residual, 2: point-mass residual
    int n_removed;
};

template <int VPT, bool VEC>
__global__ void __launch_bounds__(kScanThreads)
accept_bonus_kernel(const float* __restrict__ target_logits, long long t_stride,
                    const float* __restrict__ draft_logits_all, long long d_stride,
                    const int32_t* __restrict__ sel_index, const int32_t* __restrict__ sel_parent,
                    const int32_t* __restrict__ sel_token, const int32_t* __restrict__ n_sel,
                    const float* __restrict__ u_accept, const float* __restrict__ u_bonus, int V, int k,
                    int D, int m, int R, int chunks, float inv_t, int32_t* __restrict__ acc_len,
                    int32_t* __restrict__ acc_path, int32_t* __restrict__ bonus_token, AcceptWs ws,
                    int32_t* d_status) {
    constexpr int NE = 4 * VPT;
    __shared__ int s_par[EAGLE2_MAX_M];
    __shared__ double s_thr[EAGLE2_MAX_M];
    __shared__ float s_u[EAGLE2_MAX_M];
    __shared__ int s_walk[3];
    __shared__ int s_rtok[EAGLE2_MAX_K];
    __shared__ float s_ralpha[EAGLE2_MAX_K];
    __shared__ float s_redf[kScanWarps];
    __shared__ double s_redd[kScanWarps];
    __shared__ double s_scan[kScanThreads];
    __shared__ int s_flag, s_pick;

    const int chunk = blockIdx.x % chunks;
    const int b = blockIdx.x / chunks;
    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    chain_wait();
    chain_release();
    const int ns = min(n_sel[b], m);
    const int32_t* idx_b = sel_index + (long long)b * m;

    for (int x = tid; x < m; x += kScanThreads) {
        s_par[x] = sel_parent[(long long)b * m + x];
        s_thr[x] = ws.thr[(size_t)b * m + x];
        s_u[x] = u_accept[(long long)b * m + x];
    }
    __syncthreads();
    if (warp == 0) {
        int32_t* path = chunk == 0 ? acc_path + (long long)b * D : nullptr;
        const WalkResult w = walk_tree(s_par, s_thr, s_u, idx_b, ns, k, D, path);
        if (lane == 0) {
            s_walk[0] = w.cur, s_walk[1] = w.len, s_walk[2] = w.slot_row;
            if (chunk == 0) {
                acc_len[b] = w.len;
                for (int j = w.len; j < D; ++j) path[j] = -1;
            }
        }
    }
    __syncthreads();
    const int cur = s_walk[0], slot_row = s_walk[2];

    // ---- the distribution the extra token is drawn from -----------------------------------------
    BonusLaw law;
    law.zp = target_logits + (long long)b * t_stride + (long long)(cur + 1) * V;
    law.zq = nullptr;
    law.inv_t = inv_t;
    law.mode = 0;
    law.n_removed = 0;
    law.gmax_p = law.gmax_q = law.c_p = law.c_q = law.alpha = 0.f;
    if (slot_row >= 0) {
        const ChainSlot* slot = ws.slots + (size_t)b * R + slot_row;
        law.gmax_p = slot->gmax_p, law.c_p = slot->c_p;
        law.n_removed = slot->n_children;
        if (draft_logits_all) {
            law.mode = 1;
            law.zq = draft_logits_all + (long long)b * d_stride + (long long)slot_row * V;
            law.gmax_q = slot->gmax_q, law.c_q = slot->c_q;
            law.alpha = (float)slot->alpha;
        } else {
            law.mode = 2;
        }
        // the rejected children's tokens carry their own alpha (or are simply absent)
        if (tid < law.n_removed) {
            int c = 0, x = -1;
            for (int y = cur + 1; y < ns; ++y)
                if (s_par[y] == cur && c++ == tid) { x = y; break; }
            s_rtok[tid] = x >= 0 ? sel_token[(long long)b * m + x] : -1;
            s_ralpha[tid] = law.mode == 1 ? (float)slot->removed_alpha[tid]
                                          : (slot->removed[tid] ? INFINITY : 0.f);
        }
    }
    __syncthreads();

    auto weight_of = [&](int e, float zp_e, float zq_e, float cmax) -> float {
        if (law.mode == 0) return exp_scaled(scale_logit(zp_e, law.inv_t), cmax);
        const float pe = prob_of(zp_e, law.inv_t, law.gmax_p, law.c_p);
        float al = law.alpha;
        for (int i = 0; i < law.n_removed; ++i)
            if (s_rtok[i] == e) al = s_ralpha[i];
        if (law.mode == 2) return al == INFINITY ? 0.f : pe;
        const float qe = prob_of(zq_e, law.inv_t, law.gmax_q, law.c_q);
        return fmaxf(fmaf(-al, qe, pe), 0.f);
    };

    // ---- this chunk's total weight ----------------------------------------------------------------
    float xp[NE], xq[NE];
    scan_load<VPT, VEC>(law.zp, V, chunk, xp);
    if (law.mode == 1) scan_load<VPT, VEC>(law.zq, V, chunk, xq);
    float cmax = 0.f;
    if (law.mode == 0) {
        float t = -INFINITY;
#pragma unroll
        for (int j = 0; j < NE; ++j) t = fmaxf(t, scale_logit(xp[j], law.inv_t));
        cmax = block_max_f32(t, s_redf);
    }
    float wsum = 0.f;
    int last_pos = -1, bad = 0;
    if (law.mode != 0 || cmax > -INFINITY) {
#pragma unroll
        for (int j = 0; j < NE; ++j) {
            const int e = scan_elem_index<VPT, VEC>(chunk, j);
            if (e < V) {
                bad |= !(xp[j] < INFINITY);
                const float wgt = weight_of(e, xp[j], law.mode == 1 ? xq[j] : 0.f, cmax);
                wsum += wgt;
                if (wgt > 0.f) last_pos = max(last_pos, e);
            }
        }
    }
    const double csum = block_sum_f64((double)wsum, s_redd);
    // largest positive index of the chunk
    {
        int lp = last_pos;
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) lp = max(lp, __shfl_xor_sync(0xffffffffu, lp, o));
        __syncthreads();
        if (lane == 0) s_scan[warp] = (double)lp;
        __syncthreads();
        if (tid == 0) {
            double best = s_scan[0];
            for (int w = 1; w < kScanWarps; ++w) best = fmax(best, s_scan[w]);
            ws.blast[(size_t)b * chunks + chunk] = (int)best;
            ws.bstats[(size_t)b * chunks + chunk] = make_double2((double)cmax, csum);
        }
    }
    if (bad) raise_status(d_status, EAGLE2_STATUS_NONFINITE_LOGIT);
    if (!last_block_arrives(ws.counters + b, chunks, &s_flag)) return;

    // ---- last block: find the chunk, then the token, where the CDF passes u * total ---------------
    const double2* st = ws.bstats + (size_t)b * chunks;
    float gm = -INFINITY;
    if (law.mode == 0)
        for (int c = tid; c < chunks; c += kScanThreads) gm = fmaxf(gm, (float)st[c].x);
    const double gmax = law.mode == 0 ? (double)block_max_f32(gm, s_redf) : 0.0;
    auto chunk_weight = [&](int c) -> double {
        const double2 v = st[c];
        if (law.mode != 0) return v.y;
        return v.x > -INFINITY ? v.y * exp(v.x - gmax) : 0.0;
    };
    double part_total = 0.0;
    for (int c = tid; c < chunks; c += kScanThreads) part_total += chunk_weight(c);
    const double total = block_sum_f64(part_total, s_redd);
    const double thr_all = (double)u_bonus[b] * total;
    if (tid == 0) s_pick = -1;
    double carry_c = 0.0;
    for (int c0 = 0; c0 < chunks; c0 += kScanThreads) {
        const int c = c0 + tid;
        const double wc = c < chunks ? chunk_weight(c) : 0.0;
        __syncthreads();
        s_scan[tid] = wc;
        __syncthreads();
        for (int o = 1; o < kScanThreads; o <<= 1) {
            const double add = tid >= o ? s_scan[tid - o] : 0.0;
            __syncthreads();
            s_scan[tid] += add;
            __syncthreads();
        }
        const double incl = carry_c + s_scan[tid];
        const double span = s_scan[kScanThreads - 1];
        const bool crosses = c < chunks && incl > thr_all && (incl - wc) <= thr_all;
        __syncthreads();
        if (crosses) {  // at most one chunk: the inclusive sums are non-decreasing
            s_pick = c;
            s_scan[0] = incl - wc;  // mass before the chunk
        }
        __syncthreads();
        if (s_pick >= 0) break;
        carry_c += span;
    }
    if (tid == 0) s_scan[1] = thr_all;
    __syncthreads();
    const int pick = s_pick;
    int result = -1;
    if (pick >= 0) {
        const double before = s_scan[0], thr = s_scan[1];
        // weights of the picked chunk relative to the global maximum
        const float pmax = (float)st[pick].x;
        const double rescale = law.mode == 0 ? exp((double)pmax - gmax) : 1.0;
        __syncthreads();
        scan_load<VPT, VEC>(law.zp, V, pick, xp);
        if (law.mode == 1) scan_load<VPT, VEC>(law.zq, V, pick, xq);
        double carry = before;
        // ascending token order: for the vector layout, groups i = 0..VPT-1 of 4 consecutive tokens
        // per thread; for the scalar layout, 4*VPT groups of one token per thread
        constexpr int GROUPS = VEC ? VPT : NE;
        constexpr int PER = VEC ? 4 : 1;
        int found = 0x7fffffff;
#pragma unroll
        for (int gi = 0; gi < GROUPS; ++gi) {
            double wv[PER];
            double local = 0.0;
#pragma unroll
            for (int t = 0; t < PER; ++t) {
                const int j = gi * PER + t;
                const int e = scan_elem_index<VPT, VEC>(pick, j);
                wv[t] = e < V ? (double)weight_of(e, xp[j], law.mode == 1 ? xq[j] : 0.f, pmax) * rescale : 0.0;
                local += wv[t];
            }
            // inclusive scan of `local` over the threads of the block
            __syncthreads();
            s_scan[tid] = local;
            __syncthreads();
            for (int o = 1; o < kScanThreads; o <<= 1) {
                const double add = tid >= o ? s_scan[tid - o] : 0.0;
                __syncthreads();
                s_scan[tid] += add;
                __syncthreads();
            }
            double run = carry + s_scan[tid] - local;
            const double group_total = s_scan[kScanThreads - 1];
#pragma unroll
            for (int t = 0; t < PER; ++t) {
                const int j = gi * PER + t;
                const int e = scan_elem_index<VPT, VEC>(pick, j);
                run += wv[t];
                if (e < V && run > thr && wv[t] > 0.0) found = min(found, e);
            }
            carry += group_total;
        }
        // smallest qualifying token of the block
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) found = min(found, __shfl_xor_sync(0xffffffffu, found, o));
        __syncthreads();
        if (lane == 0) s_scan[warp] = (double)found;
        __syncthreads();
        if (tid == 0) {
            double best = s_scan[0];
            for (int w = 1; w < kScanWarps; ++w) best = fmin(best, s_scan[w]);
            result = best < 2147483647.0 ? (int)best : -1;
        }
    }
    if (tid == 0) {
        if (result < 0) {  // rounding left no token beyond the threshold: last token with weight
            for (int c = pick >= 0 ? pick : chunks - 1; c >= 0 && result < 0; --c)
                result = ws.blast[(size_t)b * chunks + c];
            if (result < 0) result = 0;
        }
        bonus_token[b] = result;
    }
}

}  // namespace eagle2

using namespace eagle2;

extern "C" int eagle2_accept(const float* target_logits, long long t_stride,
                             const float* draft_logits_all, long long d_stride,
                             const int32_t* sel_index, const int32_t* sel_parent,
                             const int32_t* sel_token, const int32_t* n_sel, int B, int V, int k, int D,
                             int m, float temperature, const float* u_accept, const float* u_bonus,
                             int32_t* acc_len, int32_t* acc_path, int32_t* bonus_token, void* ws,
                             size_t ws_bytes, int32_t* d_status, eagle2_stream_t stream) {
    if (!target_logits || !sel_index || !sel_parent || !sel_token || !n_sel || !acc_len || !acc_path ||
        !bonus_token || !d_status)
        return EAGLE2_ERR_NULL;
    if (temperature > 0.f && (!u_accept || !u_bonus)) return EAGLE2_ERR_NULL;
    if (B < 0 || V < 1 || k < 1 || k > EAGLE2_MAX_K || D < 1 || D > EAGLE2_MAX_DEPTH || m < 1 ||
        m > EAGLE2_MAX_M || !(temperature >= 0.f) || t_stride < 0 || d_stride < 0 ||
        nodes_of(k, D) > EAGLE2_MAX_NODES)
        return EAGLE2_ERR_SHAPE;
    if (!aligned(target_logits, 4) || (draft_logits_all && !aligned(draft_logits_all, 4)))
        return EAGLE2_ERR_ALIGN;
    if (B == 0) return EAGLE2_OK;
    if (!ws || !aligned(ws, kWsAlign)) return EAGLE2_ERR_WORKSPACE;
    const int R = 1 + (D - 1) * k;
    const int gvpt = greedy_vpt(B, m, V), bvpt = bonus_vpt(B, V);
    const int gchunks = scan_chunks(V, gvpt), bchunks = scan_chunks(V, bvpt);
    AcceptWs w;
    if (accept_ws_layout(B, m, R, gchunks, bchunks, ws, &w) > ws_bytes) return EAGLE2_ERR_WORKSPACE;
    cudaStream_t st = reinterpret_cast<cudaStream_t>(stream);
    const bool vec_t = aligned(target_logits, 16) && V % 4 == 0 && t_stride % 4 == 0;
    const bool vec_d = !draft_logits_all || (aligned(draft_logits_all, 16) && d_stride % 4 == 0);
    const bool vec = vec_t && vec_d;

    if (temperature == 0.f) {
        const long long blocks = (long long)B * (m + 1) * gchunks;
        if (blocks > 0x7fffffffLL) return EAGLE2_ERR_SHAPE;
#define EAGLE2_GREEDY_CASE(VPT_)                                                                         \
    case VPT_:                                                                                           \
        return launch_chained(vec_t ? accept_greedy_kernel<VPT_, true> : accept_greedy_kernel<VPT_, false>,       \
                              dim3((unsigned)blocks), dim3(kScanThreads), 0, st, 1, target_logits, t_stride,     \
                              sel_parent, sel_token, n_sel, V, D, m, gchunks, acc_len, acc_path, bonus_token, w, \
                              d_status);
        switch (gvpt) {
            EAGLE2_GREEDY_CASE(1)
            EAGLE2_GREEDY_CASE(2)
            EAGLE2_GREEDY_CASE(4)
        }
#undef EAGLE2_GREEDY_CASE
        return EAGLE2_ERR_SHAPE;
    }

    // ---- temperature > 0 --------------------------------------------------------------------------
    const float inv_t = 1.0f / temperature;
    // Cluster size.  One sequence: the smallest power of two whose vocabulary slices fit in shared
    // memory (many short slices: the chain of the root's children sets the time).  A batch has more
    // nodes than clusters fit on the device at once, so the fewest blocks that can hold the rows give
    // the most nodes in flight (V = 128256: 6 blocks instead of 8, 24 clusters instead of 18 at a time;
    // measured per call at B = 4 / 8 / 16 / 32: 55.9 -> 49.7, 96.3 -> 76.3, 192.7 -> 152.8, 346 -> 268 us;
    // 5 blocks with larger slices: 50.6 / 77.4 / 155.6 / 274 us).
    int cs = 1;
    if (B == 1) {
        while (cs < kMaxCluster && (V + cs - 1) / cs > kResidentSliceMax) cs <<= 1;
    } else {
        while (cs < kMaxCluster && (V + cs - 1) / cs > kResidentSliceMax) ++cs;
    }
    int slice = ((V + cs - 1) / cs + 3) / 4 * 4;
    const bool resident = slice <= kResidentSliceMax;
    const size_t dyn = resident ? sizeof(float) * 2 * (size_t)slice : 0;
    if ((long long)B * cs > 0x7fffffffLL || R > 65535) return EAGLE2_ERR_SHAPE;

    void (*chain)(const float*, long long, const float*, long long, const int32_t*, const int32_t*,
                  const int32_t*, const int32_t*, const float*, int, int, int, int, int, float, AcceptWs, int32_t*) =
        resident ? (vec ? accept_chain_kernel<true, true> : accept_chain_kernel<true, false>)
                 : (vec ? accept_chain_kernel<false, true> : accept_chain_kernel<false, false>);
    if (dyn > 40 * 1024 &&
        cudaFuncSetAttribute(chain, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)dyn) != cudaSuccess)
        return EAGLE2_ERR_CUDA;
    if (launch_chained(chain, dim3((unsigned)(B * cs), (unsigned)R, 1), dim3(kChainThreads), dyn, st, (unsigned)cs,
                       target_logits, t_stride, draft_logits_all, d_stride, sel_index, sel_parent, sel_token, n_sel,
                       u_accept, V, k, m, R, slice, inv_t, w, d_status) != EAGLE2_OK)
        return EAGLE2_ERR_CUDA;

    const long long blocks = (long long)B * bchunks;
    if (blocks > 0x7fffffffLL) return EAGLE2_ERR_SHAPE;
#define EAGLE2_BONUS_CASE(VPT_)                                                                          \
    case VPT_:                                                                                           \
        return launch_chained(vec ? accept_bonus_kernel<VPT_, true> : accept_bonus_kernel<VPT_, false>,           \
                              dim3((unsigned)blocks), dim3(kScanThreads), 0, st, 1, target_logits, t_stride,     \
                              draft_logits_all, d_stride, sel_index, sel_parent, sel_token, n_sel, u_accept,     \
                              u_bonus, V, k, D, m, R, bchunks, inv_t, acc_len, acc_path, bonus_token, w,         \
                              d_status);
    switch (bvpt) {
        EAGLE2_BONUS_CASE(1)
        EAGLE2_BONUS_CASE(2)
        EAGLE2_BONUS_CASE(4)
    }
#undef EAGLE2_BONUS_CASE
    return EAGLE2_ERR_SHAPE;
}
