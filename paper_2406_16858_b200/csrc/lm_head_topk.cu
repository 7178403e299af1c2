// The LM head fused with the first half of the expansion (paper Section 4.1: the draft model's
// features go through the LM head of the original LLM, and the expansion keeps the k most probable
// tokens of every row).  For many feature rows (rows = sequences x frontier size) the logits are as
// large as the weights, and writing them only to read them back once is most of the step's traffic.
// Here they never leave the SM: a block walks vocabulary tiles, the tensor pipe leaves
// logits[feature row][256 vocabulary entries] in tensor memory, and the epilogue threads fold each
// tile into their row's running maximum, sum of exponentials and k best (value, token) keys while
// the tensor pipe already works on the next tile (two accumulators).  When a block has walked its
// tiles it writes one partial per row, in the expansion's own workspace layout; a row-merge launch
// folds a row's partials into one, and the expansion's merge launch finishes the step from those.
//
// Operand roles are swapped against the plain LM head: the feature rows are the M side of
// tcgen05.mma, a vocabulary tile is its N = 256, so that a thread's tensor-memory lane is a feature
// row and its columns are that row's logits.  A block holds 128 feature rows.  Up to 128 rows: one
// block per SM (cta_group::1).  More: two blocks on one TPC form a pair (cta_group::2, M = 256),
// each holding 128 rows and copying half of every weight box, so that the weights cross from L2
// into shared memory once per pair; tensor memory then still has room for two accumulators.
//   TMA warp        streams [256 (pair: 128) vocabulary rows x 64 hidden columns] weight boxes and
//                   the matching 64 columns of the block's features (from L2) through a ring;
//   MMA warp        one lane (of the pair's first block) issues four K = 16 instructions per stage;
//                   the second block's lane tells it when that block's halves have landed;
//   8 epilogue warps two per tensor-memory lane quadrant, one for columns 0..127 and one for columns
//                   128..255 of every tile; the two halves of a row are combined at the end.
// Every wait on an mbarrier is bounded (EAGLE2_STATUS_TIMEOUT, copies drained, tensor memory freed).
#include <cuda.h>
#include <cuda_bf16.h>
#include <math.h>

#include "common.cuh"
#include "tcgen05.cuh"

namespace eagle2 {

size_t expand_partials_bytes(int B, int n_s, int chunks, int k);
bool expand_partials_layout(int B, int n_s, int chunks, int k, void* ws, size_t ws_bytes, double2** stats,
                            unsigned long long** keys);
int launch_expand_merge(int B, int V, int k, int D, int s, int chunks, int32_t* tree_token, int32_t* tree_parent,
                        double* tree_value, int32_t* frontier, void* ws, int32_t* d_status, cudaStream_t stream);
int launch_expand_row_merge(int B, int n_s, int slots, long long split_row, int chunks_lo, int chunks_hi, int k, void* ws,
                            void* ws_rows, cudaStream_t stream);

constexpr int kFzThreads = 64 + 256;  // TMA warp, MMA warp, eight epilogue warps
constexpr int kFzTileV = 256;         // vocabulary entries per tile = N of the instruction
constexpr int kFzTileK = 64;          // hidden columns per stage (128 bytes, the swizzle span)
constexpr int kFzMaxK = 16;           // keys a row's list holds (children per node the fused path supports)
constexpr int kFzMaxStages = 6;
constexpr uint32_t kFzABytes = 128 * kFzTileK * 2;  // the block's feature rows' share of a stage

struct FzBarriers {
    unsigned long long full[kFzMaxStages], empty[kFzMaxStages];
    unsigned long long peer[kFzMaxStages];  // first block of a pair: the second block's halves have landed
    unsigned long long acc_full[2], acc_empty[2];  // an accumulator is complete / has been read
    unsigned long long comb;                       // the upper column half's results are in shared memory
    unsigned long long drain;
};

__device__ __forceinline__ void fz_tma_2d(uint32_t dst, const CUtensorMap* map, int c0, int c1, uint32_t bar) {
    asm volatile(
        "cp.async.bulk.tensor.2d.shared::cta.global.tile.mbarrier::complete_tx::bytes "
        "[%0], [%1, {%2, %3}], [%4];"
        ::"r"(dst), "l"(map), "r"(c0), "r"(c1), "r"(bar)
        : "memory");
}

// A key enters a row's descending list of k: every entry it beats moves down one place, the k-th
// drops out.  All comparisons are independent of each other (no chain through the list).  Returns
// the list's k-th key afterwards (0 while the list holds fewer than k).
__device__ __forceinline__ unsigned long long fz_insert(unsigned long long (&list)[kFzMaxK], unsigned long long key, int k) {
    bool gt[kFzMaxK];
#pragma unroll
    for (int j = 0; j < kFzMaxK; ++j) gt[j] = key > list[j];
#pragma unroll
    for (int j = kFzMaxK - 1; j >= 1; --j)
        if (j < k) list[j] = gt[j] ? (gt[j - 1] ? list[j - 1] : key) : list[j];
    list[0] = gt[0] ? key : list[0];
    unsigned long long kth = 0ull;
#pragma unroll
    for (int j = 0; j < kFzMaxK; ++j)
        if (j < k) kth = list[j];  // ends as list[k - 1] (written so that the list stays in registers)
    return kth;
}

// rows: feature rows of this pass (<= 128, pair: <= 256); row0: first of them among all rows of the
// call; chunks: producers per row (= blocks or pairs of the launch); slots: partial places per row in
// stats/keys, the expansion's partial arrays (>= chunks).
template <bool PAIR>
__global__ void __launch_bounds__(kFzThreads, 1)
lm_head_topk_kernel(const __grid_constant__ CUtensorMap w_map, const __grid_constant__ CUtensorMap h_map, int rows,
                    int row0, int H, int V, int k, int stages, int chunks, int slots, long long wait_limit,
                    double2* __restrict__ stats, unsigned long long* __restrict__ keys, int32_t* d_status) {
    extern __shared__ unsigned char smem_raw[];
    __shared__ FzBarriers bars;
    __shared__ uint32_t s_tmem_base;
    __shared__ WaitCtl s_ctl;
    constexpr int CG = PAIR ? 2 : 1;
    constexpr uint32_t kBBytes = (PAIR ? kFzTileV / 2 : kFzTileV) * kFzTileK * 2;  // this block's weight box
    constexpr uint32_t kStageBytes = kFzABytes + kBBytes;
    constexpr uint32_t kTmemCols = 2 * kFzTileV;  // two accumulators: all of tensor memory

    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    const uint32_t rank = PAIR ? cluster_ctarank() : 0u;
    const int unit = PAIR ? (int)(blockIdx.x >> 1) : (int)blockIdx.x;  // walks tiles unit, unit + chunks, ...
    const uint32_t smem_base = (smem_u32(smem_raw) + 1023u) & ~1023u;
    unsigned char* smem_gen = smem_raw + (smem_base - smem_u32(smem_raw));
    const int n_tiles = (V + kFzTileV - 1) / kFzTileV;
    const int n_kb = H / kFzTileK;
    const int my_tiles = unit < n_tiles ? (n_tiles - unit + chunks - 1) / chunks : 0;
    const int rows_here = max(0, min(128, rows - (int)rank * 128));  // feature rows this block holds
    volatile WaitCtl* ctl = &s_ctl;
    long long issued = 0;  // producer lane: stages requested so far

    if (tid == 0) {
        s_ctl.abort = 0;
        s_ctl.limit = wait_limit;
        for (int s = 0; s < kFzMaxStages; ++s) {
            mbar_init(smem_u32(&bars.full[s]), 1);
            mbar_init(smem_u32(&bars.empty[s]), 1);
            mbar_init(smem_u32(&bars.peer[s]), 1);
        }
        for (int a = 0; a < 2; ++a) {
            mbar_init(smem_u32(&bars.acc_full[a]), 1);
            mbar_init(smem_u32(&bars.acc_empty[a]), 8 * CG);  // one arrival per epilogue warp of every block
        }
        mbar_init(smem_u32(&bars.comb), 4);
        mbar_init(smem_u32(&bars.drain), 1);
        fence_barrier_init();
    }
    if (warp == 1) {
        if (PAIR) {
            tmem_alloc2(smem_u32(&s_tmem_base), kTmemCols);
            tmem_relinquish2();
        } else {
            tmem_alloc(smem_u32(&s_tmem_base), kTmemCols);
            tmem_relinquish();
        }
    }
    if (warp == 0 && lane == 0) {
        asm volatile("prefetch.tensormap [%0];" ::"l"(&w_map) : "memory");
        asm volatile("prefetch.tensormap [%0];" ::"l"(&h_map) : "memory");
    }
    tc_fence_before();
    if (PAIR) cluster_sync_all();  // both blocks' barriers exist before either signals the other
    else __syncthreads();
    tc_fence_after();
    chain_wait();
    chain_release();
    const uint32_t tmem = s_tmem_base;

    if (warp == 0) {
        // ===== producer =============================================================================
        if (lane == 0) {
            bool ok = true;
            int st = 0;
            uint32_t ph = 0;
            for (int i = 0; i < my_tiles && ok; ++i) {
                const int t = unit + i * chunks;
                for (int kb = 0; kb < n_kb; ++kb, ++issued) {
                    if (issued >= stages) ok = mbar_wait_spin(smem_u32(&bars.empty[st]), ph ^ 1u, ctl);
                    if (!ok) break;
                    const uint32_t dst = smem_base + (uint32_t)st * kStageBytes;
                    const uint32_t bar = smem_u32(&bars.full[st]);
                    mbar_expect_tx(bar, kStageBytes);
                    // feature rows past the last one and vocabulary rows past V read as zero; a pair
                    // block takes its 128 of the tile's 256 vocabulary rows
                    fz_tma_2d(dst, &h_map, kb * kFzTileK, row0 + (int)rank * 128, bar);
                    fz_tma_2d(dst + kFzABytes, &w_map, kb * kFzTileK, t * kFzTileV + (int)rank * (kFzTileV / 2), bar);
                    if (++st == stages) st = 0, ph ^= 1u;
                }
            }
        }
    } else if (warp == 1) {
        // ===== MMA issuer: lane 0 alone waits and issues ================================================
        if (lane == 0) {
            int st = 0;
            uint32_t ph = 0;
            bool ok = true;
            if (PAIR && rank != 0) {
                // the second block of a pair issues nothing: it tells the first when its halves are in place
                for (long long j = 0; j < (long long)my_tiles * n_kb && ok; ++j) {
                    ok = mbar_wait_spin(smem_u32(&bars.full[st]), ph, ctl);
                    if (!ok) break;
                    mbar_arrive_in(smem_u32(&bars.peer[st]), 0);
                    if (++st == stages) st = 0, ph ^= 1u;
                }
            } else {
                constexpr uint32_t idesc = instr_desc(kFzTileV, false, PAIR ? 256 : 128);
                const uint64_t d0 = smem_desc(smem_base, 16);
                const uint32_t lo0 = (uint32_t)d0, hi = (uint32_t)(d0 >> 32);
                auto commit = [&](uint32_t bar) {
                    if (PAIR) tc_commit2(bar);
                    else tc_commit(bar);
                };
                for (int i = 0; i < my_tiles && ok; ++i) {
                    const int a = i & 1;
                    if (i >= 2) ok = mbar_wait_spin(smem_u32(&bars.acc_empty[a]), (uint32_t)(((i >> 1) - 1) & 1), ctl);
                    if (!ok) break;
                    tc_fence_after();
                    const uint32_t d_tmem = tmem + (uint32_t)a * kFzTileV;
                    for (int kb = 0; kb < n_kb; ++kb) {
                        ok = mbar_wait_spin(smem_u32(&bars.full[st]), ph, ctl);
                        if (PAIR) ok = ok && mbar_wait_spin(smem_u32(&bars.peer[st]), ph, ctl);
                        if (!ok) break;
                        tc_fence_after();
                        const uint32_t a_lo = lo0 + (uint32_t)st * (kStageBytes >> 4);
                        const uint32_t b_lo = a_lo + (kFzABytes >> 4);
                        if (kb == 0) umma_ss<CG, 0>(d_tmem, a_lo, hi, b_lo, hi, idesc);
                        else umma_ss<CG, 1>(d_tmem, a_lo, hi, b_lo, hi, idesc);
#pragma unroll
                        for (int ks = 1; ks < kFzTileK / 16; ++ks)
                            umma_ss<CG, 1>(d_tmem, a_lo + (uint32_t)ks * 2u, hi, b_lo + (uint32_t)ks * 2u, hi, idesc);
                        commit(smem_u32(&bars.empty[st]));
                        if (++st == stages) st = 0, ph ^= 1u;
                    }
                    if (ok) commit(smem_u32(&bars.acc_full[a]));
                }
            }
        }
    } else {
        // ===== epilogue warps: thread = feature row, warp = (lane quadrant, column half) ================
        // Warp w reads the tensor-memory lanes 32 * (w % 4) .. + 31; warps 2..5 take columns 0..127 of
        // every tile, warps 6..9 columns 128..255.
        constexpr float kLog2e = 1.4426950408889634f;
        const int quad = warp & 3, half = (warp - 2) >> 2;
        const int r_local = quad * 32 + lane;
        const bool row_ok = r_local < rows_here;
        const bool warp_live = quad * 32 < rows_here;  // a warp without rows only keeps the barriers going
        const uint32_t t_lane = tmem + ((uint32_t)(quad << 5) << 16) + (uint32_t)half * (kFzTileV / 2);
        float m_run = -INFINITY, s_run = 0.f;  // running maximum and sum of exp(x - maximum)
        unsigned long long list[kFzMaxK];       // the row's best keys so far, descending
#pragma unroll
        for (int j = 0; j < kFzMaxK; ++j) list[j] = 0ull;
        // Value of the k-th best once k keys are held.  Entries come in ascending token order, so one
        // that only equals it loses the tie: nothing at or below the bar can enter.
        float bar_f = -INFINITY;
        bool ok = true;
        for (int i = 0; i < my_tiles && ok; ++i) {
            const int a = i & 1;
            int r = 1;
            if (lane == 0) r = mbar_wait(smem_u32(&bars.acc_full[a]), (uint32_t)((i >> 1) & 1), ctl) ? 1 : 0;
            ok = __shfl_sync(0xffffffffu, r, 0) != 0;
            if (!ok) break;
            tc_fence_after();
            if (warp_live) {
                const int v0 = (unit + i * chunks) * kFzTileV + half * (kFzTileV / 2);
#pragma unroll 1
                for (int c0 = 0; c0 < kFzTileV / 2; c0 += 32) {
                    const int n_valid = V - (v0 + c0);  // vocabulary entries of this chunk that exist
                    if (n_valid <= 0) break;            // (uniform over the block)
                    uint32_t x[32];
                    tmem_ld32(t_lane + (uint32_t)(a * kFzTileV + c0), x);
                    tc_wait_ld(x);
                    if (n_valid < 32) {
#pragma unroll
                        for (int c = 0; c < 32; ++c)
                            if (c >= n_valid) x[c] = __float_as_uint(-INFINITY);
                    }
                    float cm0 = -INFINITY, cm1 = -INFINITY;
#pragma unroll
                    for (int c = 0; c < 32; c += 2) {
                        cm0 = fmaxf(cm0, __uint_as_float(x[c]));
                        cm1 = fmaxf(cm1, __uint_as_float(x[c + 1]));
                    }
                    const float cm = fmaxf(cm0, cm1);
                    if (cm > m_run) {
                        s_run *= ex2((m_run - cm) * kLog2e);  // 0 when nothing was summed yet
                        m_run = cm;
                    }
                    {   // a NaN or +inf logit leaves a NaN here; -inf adds nothing
                        float acc0 = 0.f, acc1 = 0.f;
                        const float nm = m_run > -INFINITY ? -m_run * kLog2e : 0.f;
#pragma unroll
                        for (int c = 0; c < 32; c += 2) {
                            acc0 += ex2(fmaf(__uint_as_float(x[c]), kLog2e, nm));
                            acc1 += ex2(fmaf(__uint_as_float(x[c + 1]), kLog2e, nm));
                        }
                        s_run += acc0 + acc1;
                    }
                    // Entries that may enter the list (rare once it has settled): a bit per entry, then one
                    // entry per lane and turn of a warp-wide loop, picked out of the registers by a select
                    // tree (indexing them by a run-time value would put the whole chunk into local memory).
                    uint32_t cand = 0u;
                    if (row_ok && cm > bar_f) {
#pragma unroll
                        for (int c = 0; c < 32; ++c)
                            if (__uint_as_float(x[c]) > bar_f) cand |= 1u << c;
                    }
                    while (__any_sync(0xffffffffu, cand != 0u)) {
                        if (cand) {
                            const int c = __ffs(cand) - 1;
                            cand &= cand - 1u;
                            uint32_t y16[16], y8[8], y4[4], y2[2];
#pragma unroll
                            for (int j = 0; j < 16; ++j) y16[j] = (c & 16) ? x[16 + j] : x[j];
#pragma unroll
                            for (int j = 0; j < 8; ++j) y8[j] = (c & 8) ? y16[8 + j] : y16[j];
#pragma unroll
                            for (int j = 0; j < 4; ++j) y4[j] = (c & 4) ? y8[4 + j] : y8[j];
#pragma unroll
                            for (int j = 0; j < 2; ++j) y2[j] = (c & 2) ? y4[2 + j] : y4[j];
                            const float f = __uint_as_float((c & 1) ? y2[1] : y2[0]);
                            if (f > bar_f) {  // the bar may have risen since the bits were set
                                const unsigned long long kth = fz_insert(list, make_key(f, (uint32_t)(v0 + c0 + c)), k);
                                if (kth) bar_f = key_value(kth);
                            }
                        }
                    }
                }
            }
            tc_fence_before();
            __syncwarp();
            if (lane == 0) {
                if (PAIR) mbar_arrive_in(smem_u32(&bars.acc_empty[a]), 0);
                else mbar_arrive(smem_u32(&bars.acc_empty[a]));
            }
        }
        // ---- the two column halves of a row become one partial ------------------------------------------
        // The ring is free: the last accumulator's completion covered every instruction that read it,
        // and every copy into it had landed before that.
        if (ok) {
            float2* c_ms = reinterpret_cast<float2*>(smem_gen);                              // [128]
            unsigned long long* c_keys = reinterpret_cast<unsigned long long*>(smem_gen + 1024);  // [kFzMaxK][128]
            if (half == 1) {
                if (row_ok) {
                    c_ms[r_local] = make_float2(m_run, s_run);
#pragma unroll
                    for (int j = 0; j < kFzMaxK; ++j)
                        if (j < k) c_keys[j * 128 + r_local] = list[j];
                }
                __syncwarp();
                if (lane == 0) mbar_arrive(smem_u32(&bars.comb));
            } else {
                int r = 1;
                if (lane == 0) r = mbar_wait(smem_u32(&bars.comb), 0, ctl) ? 1 : 0;
                ok = __shfl_sync(0xffffffffu, r, 0) != 0;
                if (ok && row_ok) {
                    const float2 o = c_ms[r_local];
                    const float m = fmaxf(m_run, o.x);
                    float sum = 0.f;
                    if (m_run > -INFINITY) sum += s_run * ex2((m_run - m) * kLog2e);
                    if (o.x > -INFINITY) sum += o.y * ex2((o.x - m) * kLog2e);
                    if (!(m_run > -INFINITY) && s_run != s_run) sum = s_run;  // NaN among nothing but -inf
                    if (!(o.x > -INFINITY) && o.y != o.y) sum = o.y;
#pragma unroll
                    for (int j = 0; j < kFzMaxK; ++j)
                        if (j < k) {
                            const unsigned long long key = c_keys[j * 128 + r_local];
                            if (key) fz_insert(list, key, k);
                        }
                    const size_t part = (size_t)(row0 + (int)rank * 128 + r_local) * slots + unit;
                    stats[part] = make_double2((double)m, (double)sum);
#pragma unroll
                    for (int j = 0; j < kFzMaxK; ++j)
                        if (j < k) keys[part * k + j] = list[j];
                    if (!(m < INFINITY) || sum != sum) raise_status(d_status, EAGLE2_STATUS_NONFINITE_LOGIT);
                }
            }
        }
    }

    // ---- teardown -----------------------------------------------------------------------------------
    // A block whose wait ran out tells its pair block (every thread that sees the flag on its way here
    // repeats the store), so that both take the same path below.
    if (PAIR && s_ctl.abort) {
        uint32_t remote;
        asm volatile("mapa.shared::cluster.u32 %0, %1, %2;" : "=r"(remote) : "r"(smem_u32(&s_ctl.abort)), "r"(rank ^ 1u));
        asm volatile("st.shared::cluster.u32 [%0], %1;" ::"r"(remote), "r"(1u) : "memory");
    }
    tc_fence_before();
    if (PAIR) cluster_sync_all();  // tensor memory is released by both blocks together
    else __syncthreads();
    tc_fence_after();
    if (s_ctl.abort) {
        // instructions issued before the wait ran out may still be reading shared memory and writing
        // tensor memory, and copies may still be on their way into the ring: both must have finished
        // before either memory is given back (fixed bound, about a second)
        if (warp == 1 && lane == 0 && rank == 0) {
            if (PAIR) tc_commit2(smem_u32(&bars.drain));
            else tc_commit(smem_u32(&bars.drain));
            mbar_drain(smem_u32(&bars.drain), 0);
        }
        if (warp == 0 && lane == 0) {
            for (long long j = issued > stages ? issued - stages : 0; j < issued; ++j)
                mbar_drain(smem_u32(&bars.full[j % stages]), (uint32_t)((j / stages) & 1));
        }
        tc_fence_before();
        if (PAIR) cluster_sync_all();
        else __syncthreads();
        tc_fence_after();
    }
    if (warp == 1) {
        if (PAIR) tmem_dealloc2(tmem, kTmemCols);
        else tmem_dealloc(tmem, kTmemCols);
    }
    if (tid == 0 && s_ctl.abort) raise_status(d_status, EAGLE2_STATUS_TIMEOUT);
    if (PAIR) cluster_sync_all();  // neither block leaves while the other may still signal it
}

static bool fz_matrix_map(CUtensorMap* map, const void* base, long long n_rows, int H, int box_rows) {
    EncodeTiledFn fn = encode_tiled_fn();
    if (!fn) return false;
    const cuuint64_t dims[2] = {(cuuint64_t)H, (cuuint64_t)n_rows};
    const cuuint64_t strides[1] = {(cuuint64_t)H * 2};
    const cuuint32_t box[2] = {(cuuint32_t)kFzTileK, (cuuint32_t)box_rows};
    const cuuint32_t estr[2] = {1, 1};
    return fn(map, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, const_cast<void*>(base), dims, strides, box, estr,
              CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
              CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

// Partials per row: one per block (pair of blocks) of the launch, a block per SM or fewer when the
// vocabulary has fewer tiles; never more than the row merge holds.
static int fz_chunks(int V, bool pair) {
    const int n_tiles = (V + kFzTileV - 1) / kFzTileV;
    int units = pair ? sm_count() / 2 : sm_count();
    if (units > 160) units = 160;
    if (units < 1) units = 1;
    return n_tiles < units ? n_tiles : units;
}

// Passes over the weights: all rows in one pass of single blocks up to 128 rows; otherwise passes of
// block pairs with 256 rows each, and the rest in a pass of its own (single blocks up to 128 rows).
struct FzPasses {
    int full;        // pair passes of 256 rows
    int rest;        // rows of the last pass (0: none)
    bool rest_pair;  // the last pass uses block pairs
    int chunks_pair, chunks_single, slots;
};
static FzPasses fz_passes(long long rows, int V) {
    FzPasses p;
    p.full = rows > 128 ? (int)(rows / 256) : 0;
    p.rest = (int)(rows - (long long)p.full * 256);
    p.rest_pair = p.rest > 128;
    p.chunks_pair = fz_chunks(V, true), p.chunks_single = fz_chunks(V, false);
    p.slots = (p.rest && !p.rest_pair) ? p.chunks_single : p.chunks_pair;
    if (p.full && p.chunks_pair > p.slots) p.slots = p.chunks_pair;
    return p;
}

// Two areas: the producers' partials (`slots` per row), then the rows' merged partials (one per row).
static size_t fz_ws_bytes(int B, int n_s, int V, int k, size_t* second) {
    const FzPasses p = fz_passes((long long)B * n_s, V);
    const size_t first = round_up(expand_partials_bytes(B, n_s, p.slots, k), kWsAlign);
    if (second) *second = first;
    return first + expand_partials_bytes(B, n_s, 1, k);
}

size_t lm_head_expand_workspace_bytes(int B, int V, int k) {
    const size_t a = fz_ws_bytes(B, 1, V, k, nullptr), b = fz_ws_bytes(B, k, V, k, nullptr);
    return a > b ? a : b;
}

template <bool PAIR>
static int fz_launch(const CUtensorMap& w_map, const CUtensorMap& h_map, int rows, int row0, int H, int V, int k, int chunks, int slots,
                     double2* stats, unsigned long long* keys, int32_t* d_status, cudaStream_t st) {
    constexpr uint32_t kStageBytes = kFzABytes + (PAIR ? kFzTileV / 2 : kFzTileV) * kFzTileK * 2;
    const int stages = PAIR ? 6 : 4;
    const size_t dyn = (size_t)stages * kStageBytes + 1024;
    if (cudaFuncSetAttribute(lm_head_topk_kernel<PAIR>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)dyn) != cudaSuccess) {
        cudaGetLastError();
        return EAGLE2_ERR_CUDA;
    }
    return launch_chained(lm_head_topk_kernel<PAIR>, dim3((unsigned)(chunks * (PAIR ? 2 : 1))), dim3(kFzThreads), dyn, st,
                          PAIR ? 2u : 1u, w_map, h_map, rows, row0, H, V, k, stages, chunks, slots, wait_limit_cycles(), stats, keys,
                          d_status);
}

}  // namespace eagle2

using namespace eagle2;

extern "C" int eagle2_lm_head_expand(const void* hidden, const void* weight, int H, int B, int V, int k, int D, int s,
                                     int32_t* tree_token, int32_t* tree_parent, double* tree_value, int32_t* frontier,
                                     void* ws, size_t ws_bytes, int32_t* d_status, eagle2_stream_t stream) {
    if (!hidden || !weight || !tree_token || !tree_parent || !tree_value || !frontier || !d_status) return EAGLE2_ERR_NULL;
    if (B < 0 || V < 1 || k < 1 || k > V || k > kFzMaxK || D < 1 || D > EAGLE2_MAX_DEPTH || s < 0 || s >= D ||
        nodes_of(k, D) > EAGLE2_MAX_NODES || H < kFzTileK || H % kFzTileK != 0)
        return EAGLE2_ERR_SHAPE;
    if (!aligned(hidden, 16) || !aligned(weight, 16) || !aligned(tree_value, 8)) return EAGLE2_ERR_ALIGN;
    if (B == 0) return EAGLE2_OK;
    const int n_s = s ? k : 1;
    const long long rows = (long long)B * n_s;
    if (rows > 0x7fffffffLL) return EAGLE2_ERR_SHAPE;
    if (!ws || !aligned(ws, kWsAlign)) return EAGLE2_ERR_WORKSPACE;
    const FzPasses p = fz_passes(rows, V);
    size_t second = 0;
    if (fz_ws_bytes(B, n_s, V, k, &second) > ws_bytes) return EAGLE2_ERR_WORKSPACE;
    void* ws_rows = static_cast<char*>(ws) + second;
    double2* stats = nullptr;
    unsigned long long* keys = nullptr;
    if (!expand_partials_layout(B, n_s, p.slots, k, ws, second, &stats, &keys)) return EAGLE2_ERR_WORKSPACE;
    CUtensorMap w_pair, w_single, h_map;
    // vocabulary rows past V and feature rows past the last one read as zero
    if (!fz_matrix_map(&w_pair, weight, V, H, kFzTileV / 2) || !fz_matrix_map(&w_single, weight, V, H, kFzTileV) ||
        !fz_matrix_map(&h_map, hidden, rows, H, 128))
        return EAGLE2_ERR_CUDA;
    cudaStream_t st = reinterpret_cast<cudaStream_t>(stream);
    int rc = EAGLE2_OK;
    for (int i = 0; i < p.full && rc == EAGLE2_OK; ++i)
        rc = fz_launch<true>(w_pair, h_map, 256, i * 256, H, V, k, p.chunks_pair, p.slots, stats, keys, d_status, st);
    if (rc == EAGLE2_OK && p.rest)
        rc = p.rest_pair ? fz_launch<true>(w_pair, h_map, p.rest, p.full * 256, H, V, k, p.chunks_pair, p.slots, stats, keys, d_status, st)
                         : fz_launch<false>(w_single, h_map, p.rest, p.full * 256, H, V, k, p.chunks_single, p.slots, stats, keys, d_status, st);
    if (rc != EAGLE2_OK) return rc;
    rc = launch_expand_row_merge(B, n_s, p.slots, (long long)p.full * 256, p.chunks_pair,
                                 p.rest_pair ? p.chunks_pair : p.chunks_single, k, ws, ws_rows, st);
    if (rc != EAGLE2_OK) return rc;
    return launch_expand_merge(B, V, k, D, s, 1, tree_token, tree_parent, tree_value, frontier, ws_rows, d_status, st);
}
