// Step 3 of the hot path: tree-masked attention of the verification pass (paper Section 4.2: each
// draft token sees the committed cache and its own ancestors only).
//
// Split-KV flash decoding on the Blackwell tensor path.  The m tree tokens of one sequence and the
// g = Hq/Hkv query heads that share a KV head are packed into M = m*g query rows, so every K/V tile
// read from HBM serves all of them.  A block owns (sequence, KV head, row block, KV split) with up
// to 256 packed rows (two 128-row UMMA tiles) and is warp specialised:
//   softmax warps  one thread per query row.  S = Q.K^T arrives in tensor memory; the thread reads
//                  its row, applies scale, tree mask and a lazily rescaled running maximum, and
//                  writes P as bf16 back into tensor memory over the scores it consumed.
//   TMA warp       streams 128-key K and V tiles (128-byte swizzled) through a ring of stages.
//   MMA warp       one thread issues tcgen05.mma: S = Q.K^T (operands in shared memory) and
//                  O += P.V (P from tensor memory, V in shared memory, MN-major), two score slots
//                  in flight so that the tensor pipe and the softmax warps overlap.
// The block writes final rows when its sequence needs a single split, otherwise an unnormalised
// fp32 partial plus (max, sum) that a merge kernel combines.
//
// Every wait on an mbarrier is bounded: when it runs out the block raises EAGLE2_STATUS_TIMEOUT,
// drains its own copies, frees its tensor memory and returns.
#include <cuda.h>
#include <cuda_bf16.h>
#include <math.h>

#include <mutex>
#include <type_traits>

#include "common.cuh"
#include "tcgen05.cuh"

namespace eagle2 {

constexpr int kTK = 128;              // keys per K/V tile = N of the Q.K^T instruction
constexpr int kRowsPerTile = 128;     // M of every tcgen05.mma
constexpr int kMaxTilesPerSplit = 16; // sequences that would need longer blocks are served longest first (batches)
constexpr int kMaxTilesPerSplitOrdered = 64;  // a block never streams more than 8192 keys
constexpr int kTmemCols = 512;
constexpr int kSlots = 2;             // score slots in tensor memory
constexpr int kSoftmaxThreads = 512;  // 16 softmax warps: four per SM sub-partition
constexpr int kAttnThreads = kSoftmaxThreads + 64;  // ... the TMA warp, the MMA warp

struct AttnPlan {
    int g, M;
    int n_rb;       // row blocks per (sequence, KV head)
    int per_tok;    // tree tokens per row block (the last may hold fewer)
    int per;        // packed rows per row block = per_tok * g
    int q_tma;      // 1: query rows arrive by TMA (g divides 128), 0: by cp.async
    int mt;         // 128-row tiles per block: 1 or 2
    int splits;     // KV splits per sequence (blocks of the launch)
    int per_split;  // K/V tiles per split
    int stages;     // K/V ring depth
    int setup_first;  // 1: blocks set up barriers and tensor memory before they wait for the preceding
                      // kernel (worth it when no block of the launch is expected to be idle)
    int pair;       // 1: two blocks (a cluster on one TPC) share every K/V tile through cta_group::2
                    // MMAs: each holds 128 of the 256 query rows, half of each K tile's keys and
                    // half of each V tile's columns
    int ordered;    // 1: a small kernel first lists the (sequence, split) items that have tiles, longest
                    // first, and blocks take their item from that list (ragged batches: the last wave
                    // is then made of the shortest blocks, and idle splits cost nothing)
    int fused_merge;  // 1 (ordered launches with several splits): the last block of a (sequence, KV head, row
                      // block) to finish combines the splits' partials itself, while other blocks still run
    size_t smem;
    long long wait_limit;  // bound of every device-side wait of the launch, in clock cycles
};

static void attention_plan(int B, int m, int Hq, int Hkv, int d, int max_kv_len, AttnPlan* p) {
    p->g = Hq / Hkv;
    p->M = m * p->g;
    // A block holds at most 256 packed rows, i.e. at most 256/g whole tokens (g need not divide 256).
    const int per_tok_max = (2 * kRowsPerTile) / p->g;
    p->n_rb = (m + per_tok_max - 1) / per_tok_max;
    p->per_tok = (m + p->n_rb - 1) / p->n_rb;
    p->per = p->per_tok * p->g;  // <= per_tok_max * g <= 256
    p->mt = p->per > kRowsPerTile ? 2 : 1;
    p->q_tma = (kRowsPerTile % p->g) == 0;
    const long long items = (long long)B * Hkv * p->n_rb;
    const int sms = sm_count(), tpcs = sms / 2;  // a pair needs both SMs of a TPC
    // Pairs pay off while the launch is short of blocks and every sequence is cut into several
    // splits (they halve the query and partial traffic); a launch that fills the device without
    // splitting is better served by independent blocks.
    // ... and while the pair's blocks stay short: with long blocks the relay between the two blocks
    // costs more per tile than the halved partials save (70B-shaped layer, 17 tiles per pair block
    // against 8 per single block: 35.6 against 34.2 us; LLaMA3-8B-shaped layer, 4 against 2: 18.5
    // against 19.7 us).
    const int tiles = (max_kv_len + m + kTK - 1) / kTK;
    p->pair = (p->mt == 2 && p->q_tma && d == 128 && items * 2 <= tpcs &&
               (tiles + tpcs / items - 1) / (tpcs / items) <= 8) ? 1 : 0;
    long long s = (p->pair ? tpcs : sms) / (items > 0 ? items : 1);
    if (s < 1) s = 1;
    if (s > tiles) s = tiles;
    int per_split = (int)((tiles + s - 1) / s);
    // a batch whose longest sequence needs several blocks anyway: order them, and let each stream more
    p->ordered = (B > 1 && !p->pair && per_split > kMaxTilesPerSplit) ? 1 : 0;
    // An ordered launch with few (sequence, KV head) items - up to one and a half per TPC - runs on
    // pairs as well: with so few items the longest sequences decide the time, and a pair puts two SMs
    // on each of their splits (measured per layer, ragged batches of the LLaMA3-8B shape: B = 8 86 ->
    // 67 us, B = 12 112 -> 104 us; with more items pairs lose: B = 16 112 -> 119 us, B = 32 181 -> 216 us).
    const bool ordered_pair = p->ordered && p->mt == 2 && p->q_tma && d == 128 && 2 * items <= 3 * tpcs;
    if (ordered_pair) p->pair = 1;
    const int units = p->pair ? tpcs : sms;  // blocks (pairs) resident at once
    if (p->ordered) {
        // Only the longest length is known here and a ragged batch holds far fewer tiles than
        // sequences x longest: aim at two blocks per SM by that count, from 8 tiles per block up to a cap
        // (long blocks leave a batch of a few sequences to a handful of SMs; short ones cost partials
        // and a block's start-up each).  Measured per layer at B = 8 / 16: 110 / 111 us with 32 tiles,
        // 105 / 121 us when aiming at four blocks per SM.
        // The more items a launch has per SM, the longer a block may be before the longest ones decide the
        // time (longer blocks: fewer partials, fewer start-ups): 32 tiles up to about one item per SM, 48
        // at two (measured per layer with caps of 32 / 40 / 48 tiles: B = 16 110 / - / 133 us, B = 20
        // 130 / 130 / 146, B = 24 148 / 142 / 149, B = 28 175 / 172 / 170, B = 32 189 / 181 / 177).
        long long cap = 16 + 18 * items / sms;
        cap = cap < 32 ? 32 : (cap > kMaxTilesPerSplitOrdered ? kMaxTilesPerSplitOrdered : cap);
        const long long want = (tiles * items + 2LL * units - 1) / (2LL * units);
        per_split = (int)(want < 8 ? 8 : (want > cap ? cap : want));
    } else if (per_split > 32) {
        per_split = 32;  // more blocks than the device holds at once: several waves
    }
    if (per_split < 1) per_split = 1;
    p->per_split = per_split;
    p->splits = (tiles + per_split - 1) / per_split;
    p->fused_merge = (p->ordered && p->splits > 1) ? 1 : 0;
    const size_t unit = (size_t)(d / 64) * kTK * 128;  // one 128-row operand tile
    int stages = (int)((220 * 1024 - p->mt * unit) / (2 * unit));
    p->stages = stages > 4 ? 4 : (stages < 2 ? 2 : stages);
    p->smem = (p->mt + 2 * (size_t)p->stages) * unit + 1024;
    p->wait_limit = wait_limit_cycles();
    p->setup_first = B == 1;  // ragged batches leave many splits without tiles: those leave at once
    if (p->pair) {  // per block: one 128-row query tile, half-size K and V stages
        p->stages = p->ordered ? 5 : 4;
        p->smem = unit + (size_t)p->stages * unit + 1024;
    }
}

struct AttnWs {
    __nv_bfloat16* o_part;  // [B][Hkv][splits][n_rb][mt*128][d], unnormalised, rounded once to bf16
    float2* ml;     // [B][Hkv][splits][n_rb][mt*128]  (reference maximum in log2 units, sum)
    uint32_t* order;  // ordered launches: [0] = items with tiles, [1 + i] = sequence * splits + split of item i
    int* tickets;     // merging launches: [B][Hkv][n_rb] arrival counters, left at zero
};

static size_t attention_ws_layout(int B, int Hkv, int d, const AttnPlan& p, void* base, AttnWs* w) {
    if (p.splits == 1 && !p.ordered) return 0;
    // every operation keeps its arrival counters (B ints) at the start of the workspace and leaves
    // them zero; everything else goes behind that region so that a shared workspace stays valid
    size_t off = round_up(sizeof(int) * (size_t)B, kWsAlign);
    char* c = static_cast<char*>(base);
    if (p.splits > 1) {
        const size_t rows = (size_t)B * Hkv * p.splits * p.n_rb * p.mt * kRowsPerTile;
        if (w) w->o_part = reinterpret_cast<__nv_bfloat16*>(c + off);
        off += round_up(rows * d * sizeof(__nv_bfloat16), kWsAlign);
        if (w) w->ml = reinterpret_cast<float2*>(c + off);
        off += round_up(rows * sizeof(float2), kWsAlign);
    }
    if (p.ordered) {
        if (w) w->order = reinterpret_cast<uint32_t*>(c + off);
        off += round_up(sizeof(uint32_t) * ((size_t)B * p.splits + 1), kWsAlign);
    }
    if (p.fused_merge) {  // (cleared by the launch's own list kernel: other operations' scratch may overlap it)
        if (w) w->tickets = reinterpret_cast<int*>(c + off);
        off += round_up(sizeof(int) * (size_t)B * Hkv * p.n_rb * (p.pair ? 2 : 1), kWsAlign);
    }
    return off;
}

size_t attention_workspace_bytes(int B, int m, int Hq, int Hkv, int d, int max_kv_len) {
    AttnPlan p;
    attention_plan(B, m, Hq, Hkv, d, max_kv_len, &p);
    return attention_ws_layout(B, Hkv, d, p, nullptr, nullptr);
}

// ---- tensor maps ---------------------------------------------------------------------------------
// K and V caches are 3-D tensors [rows][Hkv][d] of bf16; a box is 128 rows of one head and 64
// columns (128 bytes, the swizzle span).  Rows beyond the cache read as zero.
static bool make_cache_map(CUtensorMap* map, const void* base, long long rows, int Hkv, int d, int box_rows = kTK,
                           CUtensorMapL2promotion promo = CU_TENSOR_MAP_L2_PROMOTION_L2_256B) {
    EncodeTiledFn fn = encode_tiled_fn();
    if (!fn) return false;
    const cuuint64_t dims[3] = {(cuuint64_t)d, (cuuint64_t)Hkv, (cuuint64_t)rows};
    const cuuint64_t strides[2] = {(cuuint64_t)d * 2, (cuuint64_t)Hkv * d * 2};
    const cuuint32_t box[3] = {64, 1, (cuuint32_t)box_rows};
    const cuuint32_t estr[3] = {1, 1, 1};
    return fn(map, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 3, const_cast<void*>(base), dims, strides, box, estr,
              CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, promo,
              CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

// Queries [B][m][Hq][d] seen as a 4-D tensor (d, head in group, token, KV head): a box of 128/g
// tokens of one KV head lands as 128 packed rows (token-major, head in group fastest).
static bool make_query_map(CUtensorMap* map, const void* base, int B, int m, int Hq, int Hkv, int d) {
    EncodeTiledFn fn = encode_tiled_fn();
    if (!fn) return false;
    const int g = Hq / Hkv;
    const cuuint64_t dims[4] = {(cuuint64_t)d, (cuuint64_t)g, (cuuint64_t)B * m, (cuuint64_t)Hkv};
    const cuuint64_t strides[3] = {(cuuint64_t)d * 2, (cuuint64_t)Hq * d * 2, (cuuint64_t)g * d * 2};
    const cuuint32_t box[4] = {64, (cuuint32_t)g, (cuuint32_t)(kRowsPerTile / g), 1};
    const cuuint32_t estr[4] = {1, 1, 1, 1};
    return fn(map, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 4, const_cast<void*>(base), dims, strides, box, estr,
              CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
              CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

// Barrier over `nthreads` threads (named barrier `id`) that also tells every one of them whether
// all of them passed `pred`: threads about to part ways over a failed wait learn it here together.
__device__ __forceinline__ bool named_barrier_and(int id, int nthreads, bool pred) {
    uint32_t r;
    asm volatile(
        "{\n\t.reg .pred p, q;\n\tsetp.ne.b32 p, %3, 0;\n\t"
        "bar.red.and.pred q, %1, %2, p;\n\tselp.b32 %0, 1, 0, q;\n\t}"
        : "=r"(r)
        : "r"(id), "r"(nthreads), "r"((uint32_t)pred)
        : "memory");
    return r != 0;
}
__device__ __forceinline__ float max3(float a, float b, float c) {
    float r;
    asm("max.f32 %0, %1, %2, %3;" : "=f"(r) : "f"(a), "f"(b), "f"(c));
    return r;
}
// Largest raw score of a 32-column chunk (TAIL: only over the columns whose visibility bit is set).
template <bool TAIL>
__device__ __forceinline__ float chunk_rowmax(const uint32_t (&r)[32], uint32_t visw, float mx) {
    float m0 = mx, m1 = -INFINITY;
#pragma unroll
    for (int c = 0; c < 32; c += 4) {
        float a[4];
#pragma unroll
        for (int e = 0; e < 4; ++e) {
            a[e] = __uint_as_float(r[c + e]);
            if (TAIL && !((visw >> (c + e)) & 1u)) a[e] = -INFINITY;
        }
        m0 = max3(m0, a[0], a[1]);
        m1 = max3(m1, a[2], a[3]);
    }
    return fmaxf(m0, m1);
}
// p = 2^(s * scale - reference) for a chunk of NC columns, packed to NC/2 bf16 pairs; the sums of the
// unrounded probabilities accumulate in two packed registers.
template <bool TAIL, int NC>
__device__ __forceinline__ void chunk_probs(const uint32_t (&r)[NC], uint32_t visw, float2 scale2, float2 neg_ref2,
                                            float2& sum_a, float2& sum_b, uint32_t (&pk)[NC / 2]) {
#pragma unroll
    for (int c = 0; c < NC; c += 4) {
        float2 a = __ffma2_rn(make_float2(__uint_as_float(r[c]), __uint_as_float(r[c + 1])), scale2, neg_ref2);
        float2 bq = __ffma2_rn(make_float2(__uint_as_float(r[c + 2]), __uint_as_float(r[c + 3])), scale2, neg_ref2);
        if (TAIL) {
            if (!((visw >> c) & 1u)) a.x = -INFINITY;
            if (!((visw >> (c + 1)) & 1u)) a.y = -INFINITY;
            if (!((visw >> (c + 2)) & 1u)) bq.x = -INFINITY;
            if (!((visw >> (c + 3)) & 1u)) bq.y = -INFINITY;
        }
        const float2 pa = make_float2(ex2(a.x), ex2(a.y)), pb = make_float2(ex2(bq.x), ex2(bq.y));
        sum_a = __fadd2_rn(sum_a, pa);
        sum_b = __fadd2_rn(sum_b, pb);
        pk[c >> 1] = pack_bf16_alu(pa.x, pa.y);
        pk[(c >> 1) + 1] = pack_bf16_alu(pb.x, pb.y);
    }
}

// A sequence is served only if its length is within the plan and its rows lie inside the cache.
__device__ __forceinline__ bool sequence_ok(int L, long long row_base, int m, int max_kv_len, long long cache_rows) {
    return L >= 0 && L <= max_kv_len && row_base >= 0 && row_base + L + m <= cache_rows;
}

constexpr int kMaxStages = 6;  // K/V ring depth the barrier arrays allow
struct AttnBarriers {
    unsigned long long q_full;
    unsigned long long k_full[kMaxStages], k_empty[kMaxStages], v_full[kMaxStages], v_empty[kMaxStages];
    unsigned long long s_full[kSlots], p_full[kSlots];
    // Per accumulator (= score slot = item parity), two barriers used by its alternate uses: the
    // u-th P.V into accumulator e completes a phase of o_done[e][u & 1].  A waiter may skip phases (it only looks when it must rescale O, and at the
    // end); with two barriers the one it consults is never more than one phase ahead of it.
    unsigned long long o_done[2][2];
    // pair mode, used in the pair's first block: the other block's query tile / K half / V half
    // has landed (and its V tail is cleared)
    unsigned long long q_peer, k_peer[kMaxStages], v_peer[kMaxStages];
    unsigned long long v_landed, v_clean;  // the block's last V tile has landed / its rows past the sequence's last key are cleared
    unsigned long long drain;  // after a wait ran out: the tensor instructions issued so far have retired
};

// Visibility of the 128 keys of a tile that reaches past the committed cache, as four 32-bit words:
// bit c set = key0 + c is a cache key, or a tree key whose bit is set in the row's mask.
__device__ __forceinline__ void tile_visibility(unsigned long long mlo, unsigned long long mhi, int key0, int L,
                                                int n_keys, uint32_t (&vis)[4]) {
    unsigned long long lo, hi;
    const int off = key0 - L;  // tree index of column 0
    if (off >= 0) {
        if (off >= 128) lo = 0, hi = 0;
        else if (off >= 64) lo = mhi >> (off - 64), hi = 0;
        else if (off == 0) lo = mlo, hi = mhi;
        else lo = (mlo >> off) | (mhi << (64 - off)), hi = mhi >> off;
    } else {
        const int sh = -off;  // columns [0, sh) are cache keys
        if (sh >= 128) lo = ~0ull, hi = ~0ull;
        else if (sh >= 64) lo = ~0ull, hi = (sh == 64 ? 0ull : ((1ull << (sh - 64)) - 1)) | (mlo << (sh - 64));
        else lo = ((1ull << sh) - 1) | (mlo << sh), hi = (mlo >> (64 - sh)) | (mhi << sh);
    }
    const int nv = n_keys - key0;  // columns that exist at all
    if (nv < 128) {
        if (nv <= 0) lo = 0, hi = 0;
        else if (nv < 64) lo &= (1ull << nv) - 1, hi = 0;
        else if (nv > 64) hi &= (1ull << (nv - 64)) - 1;
        else hi = 0;
    }
    vis[0] = (uint32_t)lo, vis[1] = (uint32_t)(lo >> 32), vis[2] = (uint32_t)hi, vis[3] = (uint32_t)(hi >> 32);
}

// One warp combines the partials of one packed query row `pr` of (sequence b, KV head hk) that was
// computed in S_b > 1 splits: the lanes fetch the splits' (maximum, sum) pairs side by side, then
// every lane owns DH/32 columns of the row.
// PACKED: the fetched rows stay bf16 pairs until they are used - half the registers (62 against 116 per
// thread in the merge kernel, four blocks per SM instead of two), a little more work behind the loads.
template <int DH, bool PACKED = false>
__device__ __forceinline__ void merge_row(const AttnPlan& plan, const AttnWs& ws, int b, int hk, int pr, int S_b,
                                          int m, int Hq, int Hkv, __nv_bfloat16* __restrict__ out,
                                          float* __restrict__ lse) {
    const int lane = threadIdx.x & 31;
    const int g = plan.g, S = plan.splits;
    const int rb = pr / plan.per, r = pr % plan.per;
    const size_t rows_per_block = (size_t)plan.mt * kRowsPerTile;
    const size_t stride = (size_t)plan.n_rb * rows_per_block;  // rows between consecutive splits
    const size_t first = (((size_t)b * Hkv + hk) * S) * stride + rb * rows_per_block + r;
    constexpr int PER = DH / 32;  // 4 or 2 consecutive columns per lane
    float acc[PER];
#pragma unroll
    for (int e = 0; e < PER; ++e) acc[e] = 0.f;
    float l = 0.f, mmax = -INFINITY;
    // (Every load of a partial goes to L2: other SMs wrote the rows, possibly during this kernel.)
    // W partial rows are fetched before any is used: 16 when the sequence has many splits (one round
    // trip for the batch-1 layer's nine), fewer when it has few, so that short lists do not fetch the
    // same row over and over.  The first batch of rows is requested together with the splits'
    // (maximum, sum) pairs: neither address depends on the other's data.
    auto run = [&](auto width_tag) {
        constexpr int W = decltype(width_tag)::value;
        float v[PACKED ? 1 : W][PER];
        uint2 vp[PACKED ? W : 1];
        auto fetch = [&](int s0, int s1, int n) {
#pragma unroll
            for (int u = 0; u < W; ++u) {
                const int sl = min(s1 + u, n - 1);  // clamped: a repeated row gets weight 0 below
                const __nv_bfloat16* src = ws.o_part + (first + (size_t)(s0 + sl) * stride) * DH + lane * PER;
                uint2 t = make_uint2(0u, 0u);
                if (PER == 4) t = __ldcg(reinterpret_cast<const uint2*>(src));
                else t.x = __ldcg(reinterpret_cast<const uint32_t*>(src));
                if (PACKED) {
                    vp[u] = t;
                } else {
                    v[u][0] = __uint_as_float(t.x << 16), v[u][1] = __uint_as_float(t.x & 0xffff0000u);
                    if (PER == 4) v[u][PER - 2] = __uint_as_float(t.y << 16), v[u][PER - 1] = __uint_as_float(t.y & 0xffff0000u);
                }
            }
        };
        const int n0 = min(32, S_b);
        const float2 ml0 = lane < n0 ? __ldcg(ws.ml + first + (size_t)lane * stride) : make_float2(-INFINITY, 0.f);
        fetch(0, 0, n0);
        mmax = ml0.x;
        for (int s0 = 32; s0 < S_b; s0 += 32)
            if (s0 + lane < S_b) mmax = fmaxf(mmax, __ldcg(ws.ml + first + (size_t)(s0 + lane) * stride).x);
        mmax = warp_max_f32(mmax);
        for (int s0 = 0; s0 < S_b; s0 += 32) {
            const int n = min(32, S_b - s0);
            float2 ml = ml0;
            if (s0) ml = lane < n ? __ldcg(ws.ml + first + (size_t)(s0 + lane) * stride) : make_float2(-INFINITY, 0.f);
            float w = 0.f;  // weight of split s0 + lane
            if (lane < n && ml.x != -INFINITY) w = exp2f(ml.x - mmax), l += ml.y * w;
            for (int s1 = 0; s1 < n; s1 += W) {
                if (s0 || s1) fetch(s0, s1, n);
#pragma unroll
                for (int u = 0; u < W; ++u) {
                    float wu = __shfl_sync(0xffffffffu, w, min(s1 + u, 31));
                    if (s1 + u >= n) wu = 0.f;
                    // a split without visible keys leaves its partial row unwritten: never multiply it
                    if (PACKED) {
                        if (wu != 0.f) {
                            acc[0] += __uint_as_float(vp[u].x << 16) * wu;
                            acc[1] += __uint_as_float(vp[u].x & 0xffff0000u) * wu;
                            if (PER == 4) {
                                acc[PER - 2] += __uint_as_float(vp[u].y << 16) * wu;
                                acc[PER - 1] += __uint_as_float(vp[u].y & 0xffff0000u) * wu;
                            }
                        }
                    } else {
#pragma unroll
                        for (int e = 0; e < PER; ++e) acc[e] += wu != 0.f ? v[u][e] * wu : 0.f;
                    }
                }
            }
        }
    };
    if (S_b > 8) run(std::integral_constant<int, 16>{});
    else if (S_b > 4) run(std::integral_constant<int, 8>{});
    else run(std::integral_constant<int, 4>{});
    l = warp_sum_f32(l);
    const float inv = l > 0.f ? 1.f / l : 0.f;
    const int tok = pr / g, hq = hk * g + pr % g;
    __nv_bfloat16* dst = out + (((long long)b * m + tok) * Hq + hq) * DH + lane * PER;
#pragma unroll
    for (int e = 0; e < PER; e += 2)
        *reinterpret_cast<uint32_t*>(dst + e) = pack_bf16(acc[e] * inv, acc[e + 1] * inv);
    if (lse && lane == 0)
        lse[((long long)b * Hq + hq) * m + tok] = (mmax + log2f(l)) * 0.69314718055994531f;
}

// The same combination for R consecutive packed rows of one row block at once, when the sequence has
// at most SB splits (R * SB <= 16): a block that merges its 128 or 256 rows by itself has few warps and
// many rows, and one row at a time is one memory round trip per row.  Lane rr * SB + s fetches the
// (maximum, sum) pair of row rr in split s; every lane fetches its DH/32 columns of all R * SB partial
// rows before it uses any; the splits are added in the same order as in merge_row.
template <int DH, int R, int SB>
__device__ __forceinline__ void merge_rows_wide(const AttnPlan& plan, const AttnWs& ws, int b, int hk, int pr0, int n,
                                                int S_b, int m, int Hq, int Hkv, __nv_bfloat16* __restrict__ out,
                                                float* __restrict__ lse) {
    static_assert(R * SB <= 16 && (SB & (SB - 1)) == 0, "sixteen partial rows in flight per lane");
    const int lane = threadIdx.x & 31;
    const int g = plan.g, S = plan.splits;
    const int rb = pr0 / plan.per, r0 = pr0 % plan.per;
    const size_t rows_per_block = (size_t)plan.mt * kRowsPerTile;
    const size_t stride = (size_t)plan.n_rb * rows_per_block;  // rows between consecutive splits
    const size_t first = (((size_t)b * Hkv + hk) * S) * stride + rb * rows_per_block + r0;
    constexpr int PER = DH / 32;  // 4 or 2 consecutive columns per lane
    const int rr_l = lane / SB, s_l = lane % SB;
    const bool have = lane < R * SB && rr_l < n && s_l < S_b;
    const float2 ml = have ? __ldcg(ws.ml + first + rr_l + (size_t)s_l * stride) : make_float2(-INFINITY, 0.f);
    uint2 v[R][SB];
#pragma unroll
    for (int rr = 0; rr < R; ++rr)
#pragma unroll
        for (int sp = 0; sp < SB; ++sp) {
            v[rr][sp] = make_uint2(0u, 0u);
            if (rr < n && sp < S_b) {
                const __nv_bfloat16* src = ws.o_part + (first + rr + (size_t)sp * stride) * DH + lane * PER;
                if (PER == 4) v[rr][sp] = __ldcg(reinterpret_cast<const uint2*>(src));
                else v[rr][sp].x = __ldcg(reinterpret_cast<const uint32_t*>(src));
            }
        }
    float mx = ml.x;
#pragma unroll
    for (int o = SB / 2; o >= 1; o >>= 1) mx = fmaxf(mx, __shfl_xor_sync(0xffffffffu, mx, o));
    // a split without visible keys leaves its partial row unwritten: weight 0, never multiplied
    const float w = (have && ml.x != -INFINITY) ? exp2f(ml.x - mx) : 0.f;
    float lw = w != 0.f ? ml.y * w : 0.f;
#pragma unroll
    for (int o = SB / 2; o >= 1; o >>= 1) lw += __shfl_xor_sync(0xffffffffu, lw, o);
#pragma unroll
    for (int rr = 0; rr < R; ++rr) {
        if (rr >= n) break;  // uniform over the warp
        float acc[PER];
#pragma unroll
        for (int e = 0; e < PER; ++e) acc[e] = 0.f;
#pragma unroll
        for (int sp = 0; sp < SB; ++sp) {
            const float wu = __shfl_sync(0xffffffffu, w, rr * SB + sp);
            if (sp < S_b && wu != 0.f) {
                acc[0] += __uint_as_float(v[rr][sp].x << 16) * wu;
                acc[1] += __uint_as_float(v[rr][sp].x & 0xffff0000u) * wu;
                if (PER == 4) {
                    acc[PER - 2] += __uint_as_float(v[rr][sp].y << 16) * wu;
                    acc[PER - 1] += __uint_as_float(v[rr][sp].y & 0xffff0000u) * wu;
                }
            }
        }
        const float l = __shfl_sync(0xffffffffu, lw, rr * SB), mmax = __shfl_sync(0xffffffffu, mx, rr * SB);
        const float inv = l > 0.f ? 1.f / l : 0.f;
        const int pr = pr0 + rr;
        const int tok = pr / g, hq = hk * g + pr % g;
        __nv_bfloat16* dst = out + (((long long)b * m + tok) * Hq + hq) * DH + lane * PER;
#pragma unroll
        for (int e = 0; e < PER; e += 2)
            *reinterpret_cast<uint32_t*>(dst + e) = pack_bf16(acc[e] * inv, acc[e + 1] * inv);
        if (lse && lane == 0)
            lse[((long long)b * Hq + hq) * m + tok] = (mmax + log2f(l)) * 0.69314718055994531f;
    }
}

template <int DH, int MT, bool PAIR>
__global__ void __launch_bounds__(kAttnThreads, 1)
tree_attention_kernel(const __grid_constant__ CUtensorMap k_map, const __grid_constant__ CUtensorMap v_map,
                      const __grid_constant__ CUtensorMap q_map, const __nv_bfloat16* __restrict__ q, const int64_t* __restrict__ kv_off,
                      const int32_t* __restrict__ kv_len, const uint64_t* __restrict__ mask_bits, int m, int Hq,
                      int Hkv, long long cache_rows, int max_kv_len, AttnPlan plan, float scale_log2,
                      __nv_bfloat16* __restrict__ out, float* __restrict__ lse, AttnWs ws, int32_t* d_status) {
    constexpr int HALVES = DH / 64;                    // 64-column (128-byte) panels per operand tile
    constexpr uint32_t kPanel = kTK * 128;             // bytes of one panel: 128 rows x 128 bytes
    constexpr uint32_t kTile = HALVES * kPanel;
    constexpr int kTmaWarp = kSoftmaxThreads / 32, kMmaWarp = kTmaWarp + 1;
    constexpr uint32_t kIdescQK = instr_desc(kTK, false, PAIR ? 256 : 128);
    constexpr uint32_t kIdescPV = instr_desc(DH, true, PAIR ? 256 : 128);
    constexpr uint32_t kOCol = kSlots * kTK;           // first accumulator column of O
    // bytes a block holds of one K tile and of one V tile (a pair splits K by keys, V by columns)
    constexpr uint32_t kKPanel = PAIR ? kPanel / 2 : kPanel, kKTile = HALVES * kKPanel;
    constexpr uint32_t kVTile = PAIR ? kPanel : kTile;
    static_assert(!PAIR || (MT == 1 && DH == 128), "a pair block holds one 128-row tile, head_dim 128");

    extern __shared__ unsigned char smem_raw[];
    __shared__ AttnBarriers bars;
    __shared__ uint32_t s_tmem_base;
    __shared__ WaitCtl s_ctl;

    const int g = plan.g, M = plan.M, S = plan.splits, NST = plan.stages;
    const uint32_t rank = PAIR ? cluster_ctarank() : 0u;  // 0: the block that issues the pair's MMAs
    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    const uint32_t smem_base = (smem_u32(smem_raw) + 1023u) & ~1023u;
    const uint32_t sQ = smem_base;
    const uint32_t sK = sQ + MT * kTile;
    const uint32_t sV = sK + (uint32_t)NST * kKTile;
    unsigned char* smem_gen = smem_raw + (smem_base - smem_u32(smem_raw));

    // ---- set-up: barriers, tensor memory (reads nothing an earlier kernel could have written) ----
    auto set_up = [&]() {
        if (tid == 0) {
            s_ctl.abort = 0;
            s_ctl.limit = plan.wait_limit;
            mbar_init(smem_u32(&bars.q_full), plan.q_tma ? 1 : kSoftmaxThreads);
            for (int s = 0; s < kMaxStages; ++s) {
                mbar_init(smem_u32(&bars.k_full[s]), 1);
                mbar_init(smem_u32(&bars.k_empty[s]), 1);
                mbar_init(smem_u32(&bars.v_full[s]), 1);
                mbar_init(smem_u32(&bars.v_empty[s]), 1);
            }
            for (int s = 0; s < kSlots; ++s) {
                mbar_init(smem_u32(&bars.s_full[s]), 1);
                mbar_init(smem_u32(&bars.p_full[s]), (PAIR ? 2 : 1) * (kSoftmaxThreads / 64));  // one arrival per warp of the slot's group
            }
            mbar_init(smem_u32(&bars.q_peer), 1);
            for (int s = 0; s < kMaxStages; ++s) {
                mbar_init(smem_u32(&bars.k_peer[s]), 1);
                mbar_init(smem_u32(&bars.v_peer[s]), 1);
            }
            for (int s = 0; s < 4; ++s) mbar_init(smem_u32(&bars.o_done[s >> 1][s & 1]), 1);
            mbar_init(smem_u32(&bars.drain), 1);
            mbar_init(smem_u32(&bars.v_clean), 1);
            mbar_init(smem_u32(&bars.v_landed), 1);
            fence_barrier_init();
        }
        if (warp == kMmaWarp) {
            if (PAIR) {
                tmem_alloc2(smem_u32(&s_tmem_base), kTmemCols);
                tmem_relinquish2();
            } else {
                tmem_alloc(smem_u32(&s_tmem_base), kTmemCols);
                tmem_relinquish();
            }
        }
        if (warp == kTmaWarp && lane == 0) {
            asm volatile("prefetch.tensormap [%0];" ::"l"(&k_map) : "memory");
            asm volatile("prefetch.tensormap [%0];" ::"l"(&v_map) : "memory");
            if (plan.q_tma) asm volatile("prefetch.tensormap [%0];" ::"l"(&q_map) : "memory");
        }
        tc_fence_before();
        if (PAIR) cluster_sync_all();  // both blocks' barriers exist before either signals the other
        else __syncthreads();
        tc_fence_after();
    };
    // A launch for one sequence reads the sequence's length and offset before it waits for the
    // preceding kernel (the two loads then cost nothing after the wait; ~0.6 us per layer).  They are
    // final by then: the one kernel of this library that writes lengths does not let its dependents
    // start before it has completed, and a kernel that lets them start has itself waited for its
    // predecessors to complete.
    const bool early_len = plan.setup_first && !plan.ordered;
    int len_early = 0;
    long long off_early = 0;
    if (early_len) {
        const int b_early = (int)((PAIR ? blockIdx.x >> 1 : blockIdx.x) / (unsigned)(S * plan.n_rb * Hkv));
        len_early = kv_len[b_early], off_early = kv_off[b_early];
    }
    if (plan.setup_first) set_up();
    // (such a launch also works out which tiles and rows the block serves before it waits: below)
    if (!early_len) {
        chain_wait();
        chain_release();  // the merge kernel of this call (or whatever follows) may be scheduled from here on
    }

    int bid = PAIR ? blockIdx.x >> 1 : blockIdx.x;
    int split, rb, hk, b;
    if (plan.ordered) {  // item-major: the list says which (sequence, split) this block serves
        rb = bid % plan.n_rb;
        bid /= plan.n_rb;
        hk = bid % Hkv;
        const int item = bid / Hkv;
        if (item >= (int)ws.order[0]) return;  // (ordered launches set up after this point)
        const uint32_t packed = ws.order[1 + item];
        b = (int)(packed / (uint32_t)S), split = (int)(packed % (uint32_t)S);
    } else {
        split = bid % S;
        bid /= S;
        rb = bid % plan.n_rb;
        bid /= plan.n_rb;
        hk = bid % Hkv;
        b = bid / Hkv;
    }

    const int L_raw = early_len ? len_early : kv_len[b];
    const long long row_base = early_len ? off_early : kv_off[b];
    const bool overflow = !sequence_ok(L_raw, row_base, m, max_kv_len, cache_rows);
    const int L = overflow ? 0 : L_raw;
    const int n_keys = L + m;
    const int tiles = (n_keys + kTK - 1) / kTK;
    const int S_b = (tiles + plan.per_split - 1) / plan.per_split;  // splits this sequence uses
    const int t_begin = min(split * plan.per_split, tiles);
    const int nt = overflow ? 0 : min(plan.per_split, tiles - t_begin);
    const bool direct = S_b <= 1;  // a single split writes final rows

    // first packed row of this block and the rows that exist in it (the second block of a pair may
    // hold none: it still serves its halves of K and V)
    const int rows_blk = min(plan.per, M - rb * plan.per);
    const int row0 = rb * plan.per + (int)rank * 128;
    const int rows_here = PAIR ? max(0, min(128, rows_blk - (int)rank * 128)) : rows_blk;
    const size_t part_row0 = ((((size_t)b * Hkv + hk) * S + split) * plan.n_rb + rb) * (size_t)(plan.mt * 128) +
                             (size_t)rank * 128;

    if (overflow && tid == 0 && split == 0 && rb == 0 && hk == 0 && rank == 0)
        raise_status(d_status, EAGLE2_STATUS_KV_OVERFLOW);
    // a split past the sequence's last tile (never merged), or a rejected sequence: both blocks of a
    // pair take the same decision
    const bool active = nt > 0 && rows_blk > 0;
    if (early_len) {
        chain_wait();
        chain_release();
    }
    if (!plan.setup_first) {
        if (!active) return;
        set_up();
    }
    const uint32_t tmem = s_tmem_base;
    volatile WaitCtl* abort_flag = &s_ctl;
    int k_issued = 0, v_issued = 0;  // TMA lane: K and V tiles requested so far
    const int n_items = nt * MT;  // item i = (tile i / MT, row tile i % MT), score slot i % 2

    if (active) {
    if (warp == kTmaWarp) {
        // ===== TMA producer =======================================================================
        if (lane == 0) {
            bool ok = true;
            if (plan.q_tma) {
                mbar_expect_tx(smem_u32(&bars.q_full), MT * kTile);
#pragma unroll
                for (int t = 0; t < MT; ++t)
#pragma unroll
                    for (int h = 0; h < HALVES; ++h)
                        tma_load_4d(sQ + t * kTile + h * kPanel, &q_map, h * 64, 0,
                                    b * m + rb * plan.per_tok + (t + (int)rank) * (kRowsPerTile / g), hk,
                                    smem_u32(&bars.q_full));
            }
            for (int j = 0; j < nt && ok; ++j) {
                const int st = j % NST;
                const uint32_t ph = (uint32_t)((j / NST) & 1);
                const int row = (int)(row_base + (long long)(t_begin + j) * kTK);
                if (j >= NST) ok = mbar_wait(smem_u32(&bars.k_empty[st]), ph ^ 1u, abort_flag);
                if (!ok) break;
                mbar_expect_tx(smem_u32(&bars.k_full[st]), kKTile);
#pragma unroll
                for (int h = 0; h < HALVES; ++h)  // a pair block takes its 64 of the tile's 128 keys
                    tma_load_3d(sK + st * kKTile + h * kKPanel, &k_map, h * 64, hk, row + (int)rank * (kTK / 2),
                                smem_u32(&bars.k_full[st]));
                k_issued = j + 1;
                if (j >= NST) ok = mbar_wait(smem_u32(&bars.v_empty[st]), ph ^ 1u, abort_flag);
                if (!ok) break;
                mbar_expect_tx(smem_u32(&bars.v_full[st]), kVTile);
                if (PAIR) {  // all keys, this block's 64 of the 128 columns
                    tma_load_3d(sV + st * kVTile, &v_map, (int)rank * 64, hk, row, smem_u32(&bars.v_full[st]));
                } else {
#pragma unroll
                    for (int h = 0; h < HALVES; ++h)
                        tma_load_3d(sV + st * kTile + h * kPanel, &v_map, h * 64, hk, row, smem_u32(&bars.v_full[st]));
                }
                v_issued = j + 1;
            }
        }
    } else if (warp == kMmaWarp) {
        // ===== MMA issuer: lane 0 alone walks the tiles, waits and issues; nothing in its loop
        // involves the other lanes (a hand-off through the whole warp cost more than the eight
        // instructions it guards).  The other lanes have one job: the only tile of this block that can
        // reach past the sequence's last key is its last one, and rows past that key hold whatever
        // follows the sequence in the cache.  Lane 0 tells them when that V tile has landed (it follows
        // the ring's barriers phase by phase; a late joiner could not tell one use of a stage from the
        // next), they clear those rows in this block's V tile, so that a zero probability times a
        // non-finite value cannot reach O, and tell lane 0.
        const int jt = nt - 1;                                  // the block's last tile
        const int valid_t = n_keys - (t_begin + jt) * kTK;      // keys that exist in it
        const bool has_tail = valid_t < kTK;
        if (lane != 0) {
            if (has_tail) {
                const int st = jt % NST;
                if (mbar_wait(smem_u32(&bars.v_landed), 0, abort_flag)) {
                    constexpr int PANELS = PAIR ? 1 : HALVES;
                    const int chunks = (kTK - valid_t) * 8;
                    for (int idx = lane - 1; idx < chunks * PANELS; idx += 31) {
                        const int h = idx / chunks, rem = idx % chunks;
                        const int r = valid_t + rem / 8, c = rem % 8;
                        *reinterpret_cast<uint4*>(smem_gen + (sV - smem_base) + st * kVTile + h * kPanel + r * 128 +
                                                  c * 16) = make_uint4(0, 0, 0, 0);
                    }
                    fence_proxy_async();
                    __syncwarp(0xfffffffeu);
                    if (lane == 1) mbar_arrive(smem_u32(&bars.v_clean));
                }
            }
        } else {
            auto wait1 = [&](uint32_t bar, uint32_t parity) { return mbar_wait_spin(bar, parity, abort_flag); };
            bool ok = wait1(smem_u32(&bars.q_full), 0);
            if (PAIR && rank != 0) {
                // The second block of a pair issues no MMA: this lane tells the first block when this
                // block's query tile, K half and V half are in place.
                if (ok) mbar_arrive_in(smem_u32(&bars.q_peer), 0);
                int st = 0;
                uint32_t ph = 0;
                for (int j = 0; j < nt && ok; ++j) {
                    ok = wait1(smem_u32(&bars.k_full[st]), ph);
                    if (!ok) break;
                    mbar_arrive_in(smem_u32(&bars.k_peer[st]), 0);
                    ok = wait1(smem_u32(&bars.v_full[st]), ph);
                    if (ok && has_tail && j == jt) {
                        mbar_arrive(smem_u32(&bars.v_landed));
                        ok = wait1(smem_u32(&bars.v_clean), 0);
                    }
                    if (!ok) break;
                    mbar_arrive_in(smem_u32(&bars.v_peer[st]), 0);
                    if (++st == NST) st = 0, ph ^= 1u;
                }
            } else {
                if (PAIR) ok = ok && wait1(smem_u32(&bars.q_peer), 0);
                auto commit = [&](uint32_t bar) {
                    if (PAIR) tc_commit2(bar);
                    else tc_commit(bar);
                };
                // Descriptor words of the three operand layouts (low word: address and leading offset
                // in 16-byte units; high word: the layout's constants).
                constexpr int CG = PAIR ? 2 : 1;
                const uint64_t qd_first = smem_desc(sQ, 16), kd_first = smem_desc(sK, 16), vd_first = smem_desc(sV, kPanel);
                const uint32_t q_lo0 = (uint32_t)qd_first, k_lo0 = (uint32_t)kd_first, v_lo0 = (uint32_t)vd_first;
                const uint32_t qk_hi = (uint32_t)(qd_first >> 32), v_hi = (uint32_t)(vd_first >> 32);
                int k_st = 0, v_st = 0;        // ring stage of the K tile the next Q.K^T reads, of the V tile the next P.V reads
                uint32_t k_ph = 0, v_ph = 0;   // and the phases of their barriers
                // Waits and issues are separate steps: the loop below first makes sure that everything
                // the next sixteen instructions read is in place, then issues them back to back (the
                // lane's own instructions between two groups of eight - waits, commits, address
                // arithmetic - otherwise leave the tensor pipe idle for ~0.2 us each time).
                auto wait_qk = [&](int i) {   // the K tile of item i has landed (both halves of a pair)
                    if ((i & (MT - 1)) == 0) {
                        ok = ok && wait1(smem_u32(&bars.k_full[k_st]), k_ph);
                        if (PAIR) ok = ok && wait1(smem_u32(&bars.k_peer[k_st]), k_ph);
                    }
                };
                auto issue_qk = [&](int i) {  // S[slot] = Q[row tile] . K[tile]^T
                    const int t = i & (MT - 1);
                    const uint32_t d_tmem = tmem + (uint32_t)(i & 1) * kTK;
                    const uint32_t q_lo = q_lo0 + (uint32_t)t * (kTile >> 4), k_lo = k_lo0 + (uint32_t)k_st * (kKTile >> 4);
#pragma unroll
                    for (int ks = 0; ks < DH / 16; ++ks) {
                        const uint32_t qo = ((uint32_t)(ks / 4) * kPanel + (uint32_t)(ks % 4) * 32u) >> 4;
                        const uint32_t ko = ((uint32_t)(ks / 4) * kKPanel + (uint32_t)(ks % 4) * 32u) >> 4;
                        if (ks == 0) umma_ss<CG, 0>(d_tmem, q_lo + qo, qk_hi, k_lo + ko, qk_hi, kIdescQK);
                        else umma_ss<CG, 1>(d_tmem, q_lo + qo, qk_hi, k_lo + ko, qk_hi, kIdescQK);
                    }
                    commit(smem_u32(&bars.s_full[i & 1]));
                    if (t == MT - 1) {
                        commit(smem_u32(&bars.k_empty[k_st]));
                        if (++k_st == NST) k_st = 0, k_ph ^= 1u;
                    }
                };
                auto wait_pv = [&](int i) {   // the V tile of item i has landed, its probabilities are written
                    const int t = i & (MT - 1), j = MT == 1 ? i : (i >> 1);
                    if (t == 0) {
                        ok = ok && wait1(smem_u32(&bars.v_full[v_st]), v_ph);
                        if (ok && has_tail && j == jt) {
                            mbar_arrive(smem_u32(&bars.v_landed));
                            ok = wait1(smem_u32(&bars.v_clean), 0);
                        }
                        if (PAIR) ok = ok && wait1(smem_u32(&bars.v_peer[v_st]), v_ph);
                    }
                    ok = ok && wait1(smem_u32(&bars.p_full[i & 1]), (uint32_t)((i >> 1) & 1));
                };
                auto issue_pv = [&](int i) {  // O[row tile] += P[slot] . V[tile]
                    const int t = i & (MT - 1);
                    const uint32_t d_tmem = tmem + kOCol + (uint32_t)(i & 1) * DH;  // accumulator = slot = item parity
                    const uint32_t a_tmem = tmem + (uint32_t)(i & 1) * kTK;
                    const uint32_t v_lo = v_lo0 + (uint32_t)v_st * (kVTile >> 4);
#pragma unroll
                    for (int ks = 0; ks < kTK / 16; ++ks) {
                        const uint32_t vo = (uint32_t)ks * (2048u >> 4);
                        if (ks == 0) umma_ts<CG, 2>(d_tmem, a_tmem, v_lo, v_hi, kIdescPV, i >= 2 ? 1u : 0u);
                        else umma_ts<CG, 1>(d_tmem, a_tmem + ks * 16, v_lo + vo, v_hi, kIdescPV);
                    }
                    commit(smem_u32(&bars.o_done[i & 1][(i >> 1) & 1]));
                    if (t == MT - 1) {
                        commit(smem_u32(&bars.v_empty[v_st]));
                        if (++v_st == NST) v_st = 0, v_ph ^= 1u;
                    }
                };
                static_assert(kSlots == 2, "slot = item & 1");
                for (int i = 0; i < kSlots && i < n_items && ok; ++i) {
                    wait_qk(i);
                    if (!ok) break;
                    tc_fence_after();
                    issue_qk(i);
                }
                for (int i = 0; i < n_items && ok; ++i) {
                    const bool more = i + kSlots < n_items;
                    wait_pv(i);
                    if (more) wait_qk(i + kSlots);
                    if (!ok) break;
                    tc_fence_after();
                    issue_pv(i);
                    if (more) issue_qk(i + kSlots);
                }
            }
        }
        __syncwarp();
    } else {
        // ===== softmax warps: two groups of eight, each serving every other item ====================
        // A pass over one item (128 rows x 128 keys) is a chain of dependent steps - scores out of
        // tensor memory, row maximum, exchange, exponentials, probabilities back - and a group of
        // warps running it is mostly waiting; two groups on different items keep each other's
        // gaps filled.  Group e serves the items i with i % 2 == e: score slot e and accumulator e.
        // With two row tiles that is row tile e; with one row tile both groups serve it, each with
        // its own reference maximum, row sums and accumulator, and the epilogue combines the two.
        // Inside a group, warp w reads the tensor-memory lanes of its sub-partition, 32 * (w % 4) ..
        // + 31, and the two warps with the same w % 4 share 32 query rows, taking 64 of the tile's 128
        // keys each; they exchange their row maxima through shared memory behind a barrier of those 64
        // threads.  Every thread writes its probabilities over its own scores.
        __shared__ float s_xmax[2][2][2][128];            // [use parity][group][half][row]: row maxima of the halves
        __shared__ float s_xsum[2][2][128];               // epilogue: [group][half][row] row sums
        __shared__ float s_xref[2][128];                  // epilogue, one row tile: [group][row] reference maxima
        const int grp = warp >> 3, quad = warp & 3, half = (warp >> 2) & 1;
        const int r_tile = (quad << 5) | lane;            // row inside the tile = tensor-memory lane
        const uint32_t lane_sel = (uint32_t)(quad << 5) << 16;
        const int t_own = MT == 2 ? grp : 0;              // row tile this group's items belong to
        const int W = (m + 63) >> 6;
        unsigned long long mlo, mhi;
        {
            const int r_blk = t_own * 128 + r_tile;
            const int pr = r_blk < rows_here ? row0 + r_blk : rb * plan.per;  // packed row = token * g + head in group
            mlo = mask_bits[((long long)b * m + pr / g) * W];
            mhi = W > 1 ? mask_bits[((long long)b * m + pr / g) * W + 1] : 0ull;
        }
        if (!plan.q_tma) {
            // query rows into shared memory by hand, 128-byte swizzled (chunk c of row r at
            // c ^ (r & 7)); all copies of a thread are in flight together, absent rows zero-filled
#pragma unroll
            for (int it = 0; it < MT * 128 * (DH / 8) / kSoftmaxThreads; ++it) {
                const int idx = tid + it * kSoftmaxThreads;
                const int r = idx / (DH / 8), c = idx % (DH / 8);
                const bool live = r < rows_here;
                const int p2 = row0 + (live ? r : 0);
                const __nv_bfloat16* src = q + (((long long)b * m + p2 / g) * Hq + hk * g + p2 % g) * DH + c * 8;
                const int t = r >> 7, rr = r & 127, h = c >> 3, cc = c & 7;
                cp_async16(sQ + t * kTile + h * kPanel + rr * 128 + ((cc ^ (rr & 7)) << 4), src, live);
            }
            cp_async_commit();
            cp_async_wait_all();
            fence_proxy_async();
            mbar_arrive(smem_u32(&bars.q_full));
        }

        float m_ref = -INFINITY, l_run = 0.f;
        bool ok = true;
        const int pair_bar = 2 + grp * 4 + quad;  // named barrier of the two warps that share this thread's rows
        const uint32_t s_addr = tmem + lane_sel + (uint32_t)grp * kTK + (uint32_t)half * 64;  // this thread's 64 score columns
        const uint32_t o_acc = tmem + lane_sel + kOCol + (uint32_t)grp * DH;                    // this group's accumulator
        for (int i = grp; i < n_items; i += 2) {
            const int u = i >> 1;                          // the u-th use of this group's slot and accumulator
            const int j = MT == 2 ? u : i;                 // K/V tile of the item
            ok = ok && mbar_wait(smem_u32(&bars.s_full[grp]), (uint32_t)(u & 1), abort_flag);
            ok = __all_sync(0xffffffffu, ok);  // the tensor-memory accesses below need the whole warp
            const int key0 = (t_begin + j) * kTK;
            const bool tail = key0 + kTK > L;  // the tile holds tree keys or runs past the last key
            uint32_t vis0 = ~0u, vis1 = ~0u;   // visibility of this thread's keys 0..31 and 32..63
            if (tail) {
                uint32_t vis[4];
                tile_visibility(mlo, mhi, key0, L, n_keys, vis);
                vis0 = half ? vis[2] : vis[0];
                vis1 = half ? vis[3] : vis[1];
            }
            float mx = -INFINITY;
            if (ok) {
                // pass 1: the largest raw score of this thread's 64 keys (the scale is positive)
                uint32_t ba[32];
                tc_fence_after();
                tmem_ld32(s_addr, ba);
                tc_wait_ld(ba);
                mx = tail ? chunk_rowmax<true>(ba, vis0, mx) : chunk_rowmax<false>(ba, 0, mx);
                tmem_ld32(s_addr + 32, ba);
                tc_wait_ld(ba);
                mx = tail ? chunk_rowmax<true>(ba, vis1, mx) : chunk_rowmax<false>(ba, 0, mx);
                s_xmax[u & 1][grp][half][r_tile] = mx;
            }
            // the halves' maxima meet here (or both warps leave together)
            ok = named_barrier_and(pair_bar, 64, ok);
            if (!ok) break;
            mx = fmaxf(mx, s_xmax[u & 1][grp][half ^ 1][r_tile]) * scale_log2;

            // lazily rescaled reference maximum: probabilities stay below 2^8 in between.  The two
            // threads of a row hold the same reference: they derive it from the same two maxima.
            const float m_new = fmaxf(m_ref, mx);
            const bool grow = m_new > m_ref + 8.f;
            if (__any_sync(0xffffffffu, grow)) {
                const float factor = !grow ? 1.f : (m_ref == -INFINITY ? 0.f : ex2(m_ref - m_new));
                if (grow) m_ref = m_new, l_run *= factor;
                // the accumulator may be rescaled once the group's previous P.V has finished; this
                // thread owns half of the row's columns
                bool waited = true;
                if (u > 0)
                    waited = mbar_wait(smem_u32(&bars.o_done[grp][(u - 1) & 1]), (uint32_t)(((u - 1) >> 1) & 1), abort_flag);
                waited = __all_sync(0xffffffffu, waited);
                if (!waited) ok = false;  // the other warp learns it at the next barrier
                if (u > 0 && waited) {
                    tc_fence_after();
#pragma unroll
                    for (int c0 = 0; c0 < DH / 2; c0 += 32) {
                        uint32_t orow[32];
                        tmem_ld32(o_acc + (uint32_t)half * (DH / 2) + c0, orow);
                        tc_wait_ld(orow);
#pragma unroll
                        for (int c = 0; c < 32; ++c) orow[c] = __float_as_uint(__uint_as_float(orow[c]) * factor);
                        tmem_st32(o_acc + (uint32_t)half * (DH / 2) + c0, orow);
                    }
                }
            }
            // pass 2: P = 2^(s * scale - reference) as bf16.  The scores are read again, 16 keys at a
            // time, and each 16 keys become 8 packed columns written over the first half of those 16
            // score columns: no thread ever writes a column another one reads.
            const float neg_ref = m_ref == -INFINITY ? 0.f : -m_ref;
            const float2 scale2 = make_float2(scale_log2, scale_log2), neg_ref2 = make_float2(neg_ref, neg_ref);
            float2 sum_a = make_float2(0.f, 0.f), sum_b = make_float2(0.f, 0.f);
#pragma unroll
            for (int c2 = 0; c2 < 2; ++c2) {
                uint32_t b0[16], b1[16], pk[8];
                tmem_ld16(s_addr + c2 * 32, b0);
                tmem_ld16(s_addr + c2 * 32 + 16, b1);
                tc_wait_ld16(b0);
                tc_wait_ld16(b1);
                const uint32_t vw = c2 ? vis1 : vis0;
                if (tail) chunk_probs<true, 16>(b0, vw, scale2, neg_ref2, sum_a, sum_b, pk);
                else chunk_probs<false, 16>(b0, 0, scale2, neg_ref2, sum_a, sum_b, pk);
                tmem_st8(s_addr + c2 * 32, pk);
                if (tail) chunk_probs<true, 16>(b1, vw >> 16, scale2, neg_ref2, sum_a, sum_b, pk);
                else chunk_probs<false, 16>(b1, 0, scale2, neg_ref2, sum_a, sum_b, pk);
                tmem_st8(s_addr + c2 * 32 + 16, pk);
            }
            l_run += (sum_a.x + sum_a.y) + (sum_b.x + sum_b.y);
            tc_wait_st();
            tc_fence_before();
            __syncwarp();  // every lane's P is in tensor memory: one arrival speaks for the warp
            if (lane == 0) {
                if (PAIR) mbar_arrive_in(smem_u32(&bars.p_full[grp]), 0);  // the pair's first block issues P.V
                else mbar_arrive(smem_u32(&bars.p_full[grp]));
            }
        }

        // ---- epilogue: O rows leave tensor memory through shared memory, so that the global
        // stores are whole contiguous rows.  Row tile t is staged where its queries were: every
        // Q.K^T has completed once the last P.V has.  All softmax threads first agree that none of
        // them gave up.  A group that served no item (a block with a single item) contributes nothing.
        const int n_uses = (n_items - grp + 1) / 2;  // items this group served
        if (n_uses > 0)
            ok = ok && mbar_wait(smem_u32(&bars.o_done[grp][(n_uses - 1) & 1]), (uint32_t)(((n_uses - 1) >> 1) & 1), abort_flag);
        s_xsum[grp][half][r_tile] = l_run;
        if (half == 0) s_xref[grp][r_tile] = m_ref;
        ok = named_barrier_and(1, kSoftmaxThreads, ok);
        if (ok) {
            tc_fence_after();
            constexpr int NCOL = MT == 2 ? DH / 2 : DH / 4;  // columns of an output row this thread produces
            constexpr int row_bytes = DH * 2;
            const int cmask = row_bytes / 16 - 1;
            // a staged row is DH bf16; 16-byte chunk c of row r sits at chunk c ^ (r mod
            // chunks-per-row), which keeps both the row-wise writes and the chunk-wise reads free of
            // bank conflicts
            const int r_blk = t_own * 128 + r_tile;
            // One row tile: the two groups hold partial results of the same rows under their own
            // references; each thread combines a quarter of the row's columns.  Two row tiles: the
            // group's accumulator is the row tile's result and each thread takes half of the columns.
            const int col0 = MT == 2 ? half * NCOL : (2 * half + grp) * NCOL;
            float w_own = 1.f, w_oth = 0.f, l_tot, m_tot = m_ref;
            if (MT == 2) {
                l_tot = s_xsum[grp][0][r_tile] + s_xsum[grp][1][r_tile];
            } else {
                const float m0 = s_xref[0][r_tile], m1 = s_xref[1][r_tile];
                m_tot = fmaxf(m0, m1);
                const float w0 = m0 == -INFINITY ? 0.f : ex2(m0 - m_tot), w1 = m1 == -INFINITY ? 0.f : ex2(m1 - m_tot);
                l_tot = (s_xsum[0][0][r_tile] + s_xsum[0][1][r_tile]) * w0 + (s_xsum[1][0][r_tile] + s_xsum[1][1][r_tile]) * w1;
                w_own = grp ? w1 : w0, w_oth = grp ? w0 : w1;
                if (n_items < 2) w_own = grp ? 0.f : w0, w_oth = grp ? w0 : 0.f;  // accumulator 1 was never written
            }
            // final rows are normalised here; a partial stays unnormalised (the merge divides by the
            // combined sum) and is rounded to bf16 once, like a final row
            const float inv = !direct ? 1.f : (l_tot > 0.f ? 1.f / l_tot : 0.f);
            unsigned char* srow = smem_gen + t_own * kTile + (size_t)r_tile * row_bytes;
#pragma unroll
            for (int c0 = 0; c0 < NCOL; c0 += 16) {
                uint32_t oa[16], ob[16];
                tmem_ld16(o_acc + (uint32_t)(col0 + c0), oa);
                if (MT == 1) tmem_ld16(tmem + lane_sel + kOCol + (uint32_t)(grp ^ 1) * DH + (uint32_t)(col0 + c0), ob);
                tc_wait_ld16(oa);
                if (MT == 1) tc_wait_ld16(ob);
                float v[16];
#pragma unroll
                for (int c = 0; c < 16; ++c) {
                    float x = w_own != 0.f ? __uint_as_float(oa[c]) * w_own : 0.f;
                    if (MT == 1 && w_oth != 0.f) x += __uint_as_float(ob[c]) * w_oth;
                    v[c] = MT == 2 ? __uint_as_float(oa[c]) * inv : x * inv;
                }
#pragma unroll
                for (int c = 0; c < 16; c += 8) {
                    uint4 pkt;
                    pkt.x = pack_bf16(v[c + 0], v[c + 1]);
                    pkt.y = pack_bf16(v[c + 2], v[c + 3]);
                    pkt.z = pack_bf16(v[c + 4], v[c + 5]);
                    pkt.w = pack_bf16(v[c + 6], v[c + 7]);
                    const int chunk = (col0 + c0 + c) >> 3;
                    *reinterpret_cast<uint4*>(srow + (((chunk ^ r_tile) & cmask) << 4)) = pkt;
                }
            }
            if (r_blk < rows_here && half == 0 && (MT == 2 || grp == 0)) {
                const int pr = row0 + r_blk;
                if (direct) {
                    if (lse) lse[((long long)b * Hq + hk * g + pr % g) * m + pr / g] = (m_tot + log2f(l_tot)) * 0.69314718055994531f;
                } else {
                    ws.ml[part_row0 + r_blk] = make_float2(m_tot, l_tot);
                }
            }
            asm volatile("bar.sync 1, %0;" ::"n"(kSoftmaxThreads) : "memory");  // rows are staged
            const int lanes_per_row = row_bytes / 16;       // 16 lanes (8 for a 64-wide bf16 row)
            const int rows_per_pass = 32 / lanes_per_row;
            const int sub = lane / lanes_per_row, cl = lane % lanes_per_row;
            for (int r = warp * rows_per_pass + sub; r < rows_here; r += (kSoftmaxThreads / 32) * rows_per_pass) {
                const int t = r >> 7, rr = r & 127;
                const uint4 v = *reinterpret_cast<const uint4*>(smem_gen + t * kTile + (size_t)rr * row_bytes +
                                                                (((cl ^ rr) & cmask) << 4));
                if (direct) {
                    const int p2 = row0 + r;
                    __nv_bfloat16* dst = out + (((long long)b * m + p2 / g) * Hq + hk * g + p2 % g) * DH;
                    *reinterpret_cast<uint4*>(reinterpret_cast<unsigned char*>(dst) + cl * 16) = v;
                } else {
                    __nv_bfloat16* dst = ws.o_part + (part_row0 + r) * DH;
                    *reinterpret_cast<uint4*>(reinterpret_cast<unsigned char*>(dst) + cl * 16) = v;
                }
            }
        }
    }
    }  // active

    // ---- merging launches: whoever finishes a (sequence, KV head, row block) last combines its splits
    // (a pair's blocks count and merge on their own, each for its 128 rows)
    if (plan.fused_merge && !direct) {  // uniform over the block; blocks without tiles left long ago
        __shared__ int s_last;
        int* ticket = ws.tickets + (((size_t)b * Hkv + hk) * plan.n_rb + rb) * (PAIR ? 2 : 1) + rank;
        if (last_block_arrives(ticket, S_b, &s_last)) {
            constexpr int NW = kAttnThreads / 32;
            auto wide = [&](auto r_tag, auto s_tag) {
                constexpr int R = decltype(r_tag)::value, SB = decltype(s_tag)::value;
                for (int r = warp * R; r < rows_here; r += NW * R)
                    merge_rows_wide<DH, R, SB>(plan, ws, b, hk, row0 + r, min(R, rows_here - r), S_b, m, Hq, Hkv, out, lse);
            };
            if (S_b <= 2) {
                wide(std::integral_constant<int, 8>{}, std::integral_constant<int, 2>{});
            } else if (S_b <= 4) {
                wide(std::integral_constant<int, 4>{}, std::integral_constant<int, 4>{});
            } else if (S_b <= 8) {
                wide(std::integral_constant<int, 2>{}, std::integral_constant<int, 8>{});
            } else {
                for (int r = warp; r < rows_here; r += NW)
                    merge_row<DH>(plan, ws, b, hk, row0 + r, S_b, m, Hq, Hkv, out, lse);
            }
        }
    }

    // ---- teardown ----------------------------------------------------------------------------------
    // A block whose wait ran out tells its pair block (every thread that sees the flag on its way
    // here repeats the store; whoever raised it comes by after raising it), so that both take the
    // same path below.
    if (PAIR && s_ctl.abort) {
        uint32_t remote;
        asm volatile("mapa.shared::cluster.u32 %0, %1, %2;" : "=r"(remote) : "r"(smem_u32(&s_ctl.abort)), "r"(rank ^ 1u));
        asm volatile("st.shared::cluster.u32 [%0], %1;" ::"r"(remote), "r"(1u) : "memory");
        asm volatile("fence.acq_rel.cluster;" ::: "memory");  // the flag is the one thing the meeting below hands over
    }
    tc_fence_before();
    if (PAIR) cluster_sync_relaxed();  // tensor memory is released by both blocks together
    else __syncthreads();
    tc_fence_after();
    if (s_ctl.abort) {
        // Whoever gave up, and whenever: the tensor instructions issued so far may still read shared
        // memory and write tensor memory, and copies may still be on their way into the rings.  Both
        // must have finished before either memory is given back (fixed bound, about a second).
        if (warp == kMmaWarp && lane == 0 && rank == 0) {
            if (PAIR) tc_commit2(smem_u32(&bars.drain));
            else tc_commit(smem_u32(&bars.drain));
            mbar_drain(smem_u32(&bars.drain), 0);
        }
        if (warp == kTmaWarp && lane == 0) {
            if (plan.q_tma) mbar_drain(smem_u32(&bars.q_full), 0);
            for (int j = max(0, k_issued - NST); j < k_issued; ++j)
                mbar_drain(smem_u32(&bars.k_full[j % NST]), (uint32_t)((j / NST) & 1));
            for (int j = max(0, v_issued - NST); j < v_issued; ++j)
                mbar_drain(smem_u32(&bars.v_full[j % NST]), (uint32_t)((j / NST) & 1));
        }
        tc_fence_before();
        if (PAIR) cluster_sync_all();
        else __syncthreads();
        tc_fence_after();
    }
    if (warp == kMmaWarp) {
        if (PAIR) tmem_dealloc2(tmem, kTmemCols);
        else tmem_dealloc(tmem, kTmemCols);
    }
    if (tid == 0 && s_ctl.abort) raise_status(d_status, EAGLE2_STATUS_TIMEOUT);
    if (PAIR) cluster_sync_relaxed();  // neither block leaves while the other may still signal it
}

// Ordered launches: one block lists the (sequence, split) items that have tiles, most tiles first
// (a counting sort over the tile counts; the order among equals is whatever the atomics give, which
// changes nothing but the schedule).
__global__ void __launch_bounds__(1024)
tree_attention_schedule_kernel(const int64_t* __restrict__ kv_off, const int32_t* __restrict__ kv_len, int B, int m,
                               long long cache_rows, int max_kv_len, AttnPlan plan, uint32_t* __restrict__ order,
                               int* __restrict__ tickets, int n_tickets) {
    __shared__ int s_bin[kMaxTilesPerSplitOrdered + 1];  // per tile count: items, then the next free place
    chain_wait();
    chain_release();
    // the merging blocks' arrival counters start at zero whatever shared this workspace since
    for (int i = threadIdx.x; i < n_tickets; i += blockDim.x) tickets[i] = 0;
    const int S = plan.splits;
    const long long n = (long long)B * S;
    for (int i = threadIdx.x; i <= kMaxTilesPerSplitOrdered; i += blockDim.x) s_bin[i] = 0;
    __syncthreads();
    auto tiles_of = [&](long long item) {
        const int b = (int)(item / S), split = (int)(item % S);
        const int L = kv_len[b];
        if (!sequence_ok(L, kv_off[b], m, max_kv_len, cache_rows)) return 0;
        const int tiles = (L + m + kTK - 1) / kTK;
        return max(0, min(plan.per_split, tiles - split * plan.per_split));
    };
    for (long long i = threadIdx.x; i < n; i += blockDim.x) atomicAdd(&s_bin[tiles_of(i)], 1);
    __syncthreads();
    if (threadIdx.x == 0) {
        int at = 0;
        for (int t = kMaxTilesPerSplitOrdered; t >= 1; --t) {
            const int c = s_bin[t];
            s_bin[t] = at;
            at += c;
        }
        order[0] = (uint32_t)at;
    }
    __syncthreads();
    for (long long i = threadIdx.x; i < n; i += blockDim.x) {
        const int t = tiles_of(i);
        if (t > 0) order[1 + atomicAdd(&s_bin[t], 1)] = (uint32_t)i;
    }
}

// One warp per output row of a sequence that used several splits (launches that do not merge inside
// the attention kernel).
template <int DH, bool PACKED>
__global__ void __launch_bounds__(256)
tree_attention_merge_kernel(const int64_t* __restrict__ kv_off, const int32_t* __restrict__ kv_len, int B, int m,
                            int Hq, int Hkv, long long cache_rows, int max_kv_len, AttnPlan plan, AttnWs ws, __nv_bfloat16* __restrict__ out,
                            float* __restrict__ lse) {
    const long long total = (long long)B * Hkv * plan.M;
    const long long warps = ((long long)gridDim.x * blockDim.x) >> 5;
    const long long row_first = ((long long)blockIdx.x * blockDim.x + threadIdx.x) >> 5;
    // The sequence lengths are final before this kernel can start (the attention kernel lets its
    // dependents in only after its own predecessors are complete, and does not write them): the
    // first row's are read while the attention kernel is still running.
    int len_first = 0;
    long long off_first = 0;
    int pr = 0, hk = 0, b = 0;
    auto decode = [&](long long row) {
        pr = (int)(row % plan.M);
        hk = (int)((row / plan.M) % Hkv);
        b = (int)(row / ((long long)plan.M * Hkv));
    };
    if (row_first < total) {  // ... and so is the arithmetic that says which row that is
        decode(row_first);
        len_first = kv_len[b], off_first = kv_off[b];
    }
    chain_wait();  // the attention kernel's partials are complete
    chain_release();
    // a large batch is walked by a grid of a few blocks per SM: most rows need no merge
    for (long long row = row_first; row < total; row += warps) {
        if (row != row_first) decode(row);
        const int L = row == row_first ? len_first : kv_len[b];
        if (!sequence_ok(L, row == row_first ? off_first : kv_off[b], m, max_kv_len, cache_rows)) continue;
        const int tiles = (L + m + kTK - 1) / kTK;
        const int S_b = (tiles + plan.per_split - 1) / plan.per_split;
        if (S_b <= 1) continue;  // the attention kernel wrote these rows itself
        merge_row<DH, PACKED>(plan, ws, b, hk, pr, S_b, m, Hq, Hkv, out, lse);
    }
}

template <int DH, int MT, bool PAIR>
static int launch_attention(const CUtensorMap& k_map, const CUtensorMap& v_map, const CUtensorMap& q_map,
                            const void* q,
                            const int64_t* kv_off, const int32_t* kv_len, const uint64_t* mask_bits, int B,
                            int m, int Hq, int Hkv, long long cache_rows, int max_kv_len, const AttnPlan& plan,
                            float scale, void* out, float* lse, const AttnWs& ws, int32_t* d_status,
                            cudaStream_t st) {
    auto kern = tree_attention_kernel<DH, MT, PAIR>;
    if (cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)plan.smem) !=
        cudaSuccess) {
        cudaGetLastError();
        return EAGLE2_ERR_CUDA;
    }
    const long long blocks = (long long)B * Hkv * plan.n_rb * plan.splits * (PAIR ? 2 : 1);
    if (blocks > 0x7fffffffLL || (long long)B * plan.splits > 0x7fffffffLL) return EAGLE2_ERR_SHAPE;
    if (plan.ordered &&
        launch_chained(tree_attention_schedule_kernel, dim3(1), dim3(1024), 0, st, 1, kv_off, kv_len, B, m, cache_rows,
                       max_kv_len, plan, ws.order, ws.tickets, plan.fused_merge ? B * Hkv * plan.n_rb * (plan.pair ? 2 : 1) : 0) != EAGLE2_OK)
        return EAGLE2_ERR_CUDA;
    if (launch_chained(kern, dim3((unsigned)blocks), dim3(kAttnThreads), plan.smem, st, PAIR ? 2u : 1u, k_map, v_map, q_map,
                       static_cast<const __nv_bfloat16*>(q), kv_off, kv_len, mask_bits, m, Hq, Hkv, cache_rows, max_kv_len,
                       plan, scale * 1.4426950408889634f, static_cast<__nv_bfloat16*>(out), lse, ws, d_status) != EAGLE2_OK)
        return EAGLE2_ERR_CUDA;
    if (plan.splits > 1 && !plan.fused_merge) {
        const long long warps = (long long)B * Hkv * plan.M;
        long long mblocks = (warps + 7) / 8;
        if (mblocks > 8LL * sm_count()) mblocks = 8LL * sm_count();
        // Two of the merge kernel's blocks fit on an SM, four of its packed variant's.  A launch that two
        // per SM can hold runs the first (LLaMA3-8B-shaped layer, 240 blocks: 16.7 us per layer against
        // 17.1 packed and kept to two per SM, 17.8 four per SM: the blocks then sit four deep on the SMs
        // the attention blocks left first); a larger one runs the packed variant so that it is resident
        // at once (70B-shaped layer, 480 blocks: 32.7 -> 31.4 us per layer).
        const bool packed = mblocks > 2LL * sm_count();
        auto merge = packed ? tree_attention_merge_kernel<DH, true> : tree_attention_merge_kernel<DH, false>;
        if (launch_chained(merge, dim3((unsigned)mblocks), dim3(256), 0, st, 1, kv_off, kv_len, B, m,
                           Hq, Hkv, cache_rows, max_kv_len, plan, ws, static_cast<__nv_bfloat16*>(out), lse) != EAGLE2_OK)
            return EAGLE2_ERR_CUDA;
    }
    return EAGLE2_OK;
}

}  // namespace eagle2

using namespace eagle2;

extern "C" int eagle2_tree_attention_launches(int B, int m, int Hq, int Hkv, int d, int max_kv_len) {
    if (B < 1 || m < 1 || m > EAGLE2_MAX_M || Hq < 1 || Hkv < 1 || Hq % Hkv || Hq / Hkv > 8 || (d != 64 && d != 128) ||
        max_kv_len < 0)
        return 0;
    AttnPlan plan;
    attention_plan(B, m, Hq, Hkv, d, max_kv_len, &plan);
    return 1 + (plan.ordered ? 1 : 0) + ((plan.splits > 1 && !plan.fused_merge) ? 1 : 0);
}

extern "C" int eagle2_tree_attention(const void* q, const void* k_cache, const void* v_cache,
                                     long long cache_rows, const int64_t* kv_off, const int32_t* kv_len,
                                     const uint64_t* mask_bits, int B, int m, int Hq, int Hkv, int d,
                                     int max_kv_len, float scale, void* out, float* lse, void* ws,
                                     size_t ws_bytes, int32_t* d_status, eagle2_stream_t stream) {
    if (!q || !k_cache || !v_cache || !kv_off || !kv_len || !mask_bits || !out || !d_status)
        return EAGLE2_ERR_NULL;
    if (B < 0 || m < 1 || m > EAGLE2_MAX_M || Hq < 1 || Hkv < 1 || Hq % Hkv || Hq / Hkv > 8 ||
        (d != 64 && d != 128) || max_kv_len < 0 || cache_rows < 1 || cache_rows > 0x7fffffffLL ||
        (long long)max_kv_len + m > cache_rows || !(scale > 0.f))
        return EAGLE2_ERR_SHAPE;
    if (!aligned(q, 16) || !aligned(k_cache, 16) || !aligned(v_cache, 16) || !aligned(out, 16) ||
        !aligned(mask_bits, 8))
        return EAGLE2_ERR_ALIGN;
    if (B == 0) return EAGLE2_OK;
    AttnPlan plan;
    attention_plan(B, m, Hq, Hkv, d, max_kv_len, &plan);
    if (plan.per > plan.mt * kRowsPerTile || plan.per_tok * plan.n_rb < m) return EAGLE2_ERR_SHAPE;  // (cannot happen)
    AttnWs w = {nullptr, nullptr, nullptr, nullptr};
    if (plan.splits > 1 || plan.ordered) {
        if (!ws || !aligned(ws, kWsAlign)) return EAGLE2_ERR_WORKSPACE;
        if (attention_ws_layout(B, Hkv, d, plan, ws, &w) > ws_bytes) return EAGLE2_ERR_WORKSPACE;
        if ((plan.ordered && !w.order) || (plan.fused_merge && !w.tickets)) return EAGLE2_ERR_WORKSPACE;
    }
    CUtensorMap k_map, v_map, q_map;
    // a pair block loads 64 keys of every K tile (and all 128 keys of 64 V columns)
    if (!make_cache_map(&k_map, k_cache, cache_rows, Hkv, d, plan.pair ? kTK / 2 : kTK) ||
        !make_cache_map(&v_map, v_cache, cache_rows, Hkv, d, kTK,
                        plan.pair ? CU_TENSOR_MAP_L2_PROMOTION_L2_128B : CU_TENSOR_MAP_L2_PROMOTION_L2_256B))
        return EAGLE2_ERR_CUDA;
    if (plan.q_tma) {
        if (!make_query_map(&q_map, q, B, m, Hq, Hkv, d)) return EAGLE2_ERR_CUDA;
    } else {
        q_map = k_map;  // unused by the kernel
    }
    cudaStream_t st = reinterpret_cast<cudaStream_t>(stream);
#define EAGLE2_ATTN_CASE(DH_, MT_, PAIR_)                                                                       \
    return launch_attention<DH_, MT_, PAIR_>(k_map, v_map, q_map, q, kv_off, kv_len, mask_bits, B, m, Hq, Hkv,      \
                                             cache_rows, max_kv_len, plan, scale, out, lse, w, d_status, st)
    if (d == 64) {
        if (plan.mt == 1) EAGLE2_ATTN_CASE(64, 1, false);
        EAGLE2_ATTN_CASE(64, 2, false);
    }
    if (plan.pair) EAGLE2_ATTN_CASE(128, 1, true);
    if (plan.mt == 1) EAGLE2_ATTN_CASE(128, 1, false);
    EAGLE2_ATTN_CASE(128, 2, false);
#undef EAGLE2_ATTN_CASE
}
