// The LM head fused with the first half of the expansion (paper Section 4.1: the draft model's
// features go through the LM head of the original LLM, and the expansion keeps the k most probable
// tokens of every row).  For many feature rows (rows = sequences x frontier size) the logits are as
// large as the weights, and writing them only to read them back once is most of the step's traffic.
// Here they never leave the SM: a block walks tiles of 128 vocabulary entries, the tensor pipe leaves
// logits[vocabulary entry][feature row] in tensor memory, writer warps turn 32 rows at a time through
// shared memory, and scanner threads - one per feature row - fold them into the row's running
// maximum, sum of exponentials and k best (value, token) keys while the tensor pipe already works on
// the next tile (two accumulators).  When a block has walked its tiles it writes one partial per row,
// in the expansion's own workspace layout; a row-merge launch folds a row's partials into one, and the
// expansion's merge launch finishes the step from those.
//
// The vocabulary is the M side of tcgen05.mma (128 entries per block) and the feature rows are its
// N side, N = the rows of the pass rounded up to 16: the tensor work is proportional to the rows
// (with the rows on the M side it was padded to 128 or 256, which at 160 rows made it as long as the
// weight stream).  Up to 128 rows: one block per SM (cta_group::1).  More: two blocks on one TPC form
// a pair (cta_group::2, M = 256 vocabulary entries), each copying half of the feature rows, so that
// the features cross from L2 into shared memory once per pair.
//   TMA warp         streams [128 vocabulary rows x 64 hidden columns] weight boxes and the matching
//                    64 columns of the block's feature rows (from L2) through a ring;
//   MMA warp         one lane (of the pair's first block) issues four K = 16 instructions per stage;
//                    the second block's lane tells it when that block's boxes have landed;
//   4 writer warps   one per tensor-memory lane quadrant: 32 feature rows (columns) of the finished
//                    accumulator at a time into one of two shared-memory buffers, transposed
//                    ([row][vocabulary entry], rows 129 words apart: no bank conflicts either way);
//   8 scanner warps  warp c owns feature rows 32c .. 32c+31 of the pass, a thread one row.
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

constexpr int kFzWriterWarps = 4, kFzScanWarps = 8;
constexpr int kFzThreads = (2 + kFzWriterWarps + kFzScanWarps) * 32;
constexpr int kFzTileV = 128;   // vocabulary entries per block and tile = the block's M
constexpr int kFzTileK = 64;    // hidden columns per stage (128 bytes, the swizzle span)
constexpr int kFzMaxK = 16;     // keys a row's list holds (children per node the fused path supports)
constexpr int kFzMaxRows = 256; // feature rows per pass = N of the instruction at most
constexpr int kFzMaxStages = 8;
constexpr uint32_t kFzABytes = kFzTileV * kFzTileK * 2;     // the weight box of a stage
constexpr int kFzTStride = 33;                              // words between rows of a transposition unit
constexpr uint32_t kFzTBytes = 32 * kFzTStride * 4;         // one unit: 32 feature rows x 32 vocabulary entries

struct FzBarriers {
    unsigned long long full[kFzMaxStages], empty[kFzMaxStages];
    unsigned long long peer[kFzMaxStages];  // first block of a pair: the second block's boxes have landed
    unsigned long long acc_full[2], acc_empty[2];  // an accumulator is complete / has been read
    // unit (c, q) = feature rows 32c.., vocabulary entries 32q.. of the tile: written / scanned
    unsigned long long t_full[kFzScanWarps][4], t_empty[kFzScanWarps][4];
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

// rows: feature rows of this pass (<= 128, pair: <= 256); n_pad: rows rounded up to 16 (= N); row0:
// first of them among all rows of the call; units: blocks (pairs) of the launch, unit u walks tiles
// u, u + units, ...; slots: partial places per row in stats/keys, the expansion's partial arrays
// (a block writes place blockIdx.x); b_bytes: bytes of the block's feature box of a stage.
template <bool PAIR>
__global__ void __launch_bounds__(kFzThreads, 1)
lm_head_topk_kernel(const __grid_constant__ CUtensorMap w_map, const __grid_constant__ CUtensorMap h_map, int rows,
                    int n_pad, int row0, int H, int V, int k, int stages, int t_slots, int units, int slots, uint32_t b_bytes,
                    long long wait_limit, double2* __restrict__ stats, unsigned long long* __restrict__ keys,
                    int32_t* d_status) {
    extern __shared__ unsigned char smem_raw[];
    __shared__ FzBarriers bars;
    __shared__ uint32_t s_tmem_base;
    __shared__ WaitCtl s_ctl;
    constexpr int CG = PAIR ? 2 : 1;
    constexpr uint32_t kTmemCols = 2 * kFzMaxRows;  // two accumulators: all of tensor memory

    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    const uint32_t rank = PAIR ? cluster_ctarank() : 0u;
    const int unit = PAIR ? (int)(blockIdx.x >> 1) : (int)blockIdx.x;
    const uint32_t smem_base = (smem_u32(smem_raw) + 1023u) & ~1023u;
    unsigned char* smem_gen = smem_raw + (smem_base - smem_u32(smem_raw));
    const uint32_t stage_bytes = kFzABytes + b_bytes;
    float* t_buf = reinterpret_cast<float*>(smem_gen + (size_t)stages * stage_bytes);  // [chunk][t_slots][32][kFzTStride]
    const int tile_v = CG * kFzTileV;  // vocabulary entries of a tile of the unit
    const int n_tiles = (V + tile_v - 1) / tile_v;
    const int n_kb = H / kFzTileK;
    const int my_tiles = unit < n_tiles ? (n_tiles - unit + units - 1) / units : 0;
    const int n_chunks = (rows + 31) / 32;  // groups of 32 feature rows = scanner warps with work
    const int b_rows = PAIR ? n_pad / 2 : n_pad;  // feature rows this block copies
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
            mbar_init(smem_u32(&bars.acc_empty[a]), kFzWriterWarps * CG);  // one arrival per writer warp of every block
        }
        for (int c = 0; c < kFzScanWarps; ++c)
            for (int q = 0; q < 4; ++q) {
                mbar_init(smem_u32(&bars.t_full[c][q]), 1);
                mbar_init(smem_u32(&bars.t_empty[c][q]), 1);
            }
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
                // this block's 128 vocabulary rows of the tile; rows past V read as zero, and so do
                // feature rows past the call's last one
                const int vrow = (unit + i * units) * tile_v + (int)rank * kFzTileV;
                for (int kb = 0; kb < n_kb; ++kb, ++issued) {
                    if (issued >= stages) ok = mbar_wait_spin(smem_u32(&bars.empty[st]), ph ^ 1u, ctl);
                    if (!ok) break;
                    const uint32_t dst = smem_base + (uint32_t)st * stage_bytes;
                    const uint32_t bar = smem_u32(&bars.full[st]);
                    mbar_expect_tx(bar, stage_bytes);
                    fz_tma_2d(dst, &w_map, kb * kFzTileK, vrow, bar);
                    fz_tma_2d(dst + kFzABytes, &h_map, kb * kFzTileK, row0 + (int)rank * b_rows, bar);
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
                // the second block of a pair issues nothing: it tells the first when its boxes are in place
                for (long long j = 0; j < (long long)my_tiles * n_kb && ok; ++j) {
                    ok = mbar_wait_spin(smem_u32(&bars.full[st]), ph, ctl);
                    if (!ok) break;
                    mbar_arrive_in(smem_u32(&bars.peer[st]), 0);
                    if (++st == stages) st = 0, ph ^= 1u;
                }
            } else {
                const uint32_t idesc = instr_desc(n_pad, false, PAIR ? 256 : 128);
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
                    const uint32_t d_tmem = tmem + (uint32_t)a * kFzMaxRows;
                    for (int kb = 0; kb < n_kb; ++kb) {
                        ok = mbar_wait_spin(smem_u32(&bars.full[st]), ph, ctl);
                        if (PAIR) ok = ok && mbar_wait_spin(smem_u32(&bars.peer[st]), ph, ctl);
                        if (!ok) break;
                        tc_fence_after();
                        const uint32_t a_lo = lo0 + (uint32_t)st * (stage_bytes >> 4);
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
    } else if (warp < 2 + kFzWriterWarps) {
        // ===== writer warps: thread = vocabulary entry (tensor-memory lane) ==============================
        // Warp q reads the lanes 32q .. 32q+31 (q = warp % 4).  Columns 32c .. 32c+31 of the accumulator
        // are the logits of feature rows 32c .. for this thread's entry: unit (c, q), which goes to
        // slot q % t_slots of scanner warp c as [row][entry].  The slot's previous occupant is the unit
        // t_slots quadrants back - of the same tile, or of the tile before - and this warp has waited for
        // every earlier release of that unit, so the phase it looks at cannot be mistaken for another.
        const int q = warp & 3;
        const uint32_t t_lane = tmem + ((uint32_t)(q << 5) << 16);
        const int q_prev = (q + 4 - t_slots) & 3;      // the quadrant whose unit held the slot before
        const int tile_back = q < t_slots ? 1 : 0;     // ... in the tile before this one
        bool ok = true;
        for (int i = 0; i < my_tiles && ok; ++i) {
            const int a = i & 1;
            int r = 1;
            if (lane == 0) r = mbar_wait(smem_u32(&bars.acc_full[a]), (uint32_t)((i >> 1) & 1), ctl) ? 1 : 0;
            ok = __shfl_sync(0xffffffffu, r, 0) != 0;
            if (!ok) break;
            tc_fence_after();
#pragma unroll 1
            for (int c = 0; c < n_chunks; ++c) {
                uint32_t x[32];
                tmem_ld32(t_lane + (uint32_t)(a * kFzMaxRows + c * 32), x);
                if (i - tile_back >= 0) {
                    r = 1;
                    if (lane == 0)
                        r = mbar_wait(smem_u32(&bars.t_empty[c][q_prev]), (uint32_t)((i - tile_back) & 1), ctl) ? 1 : 0;
                    ok = __shfl_sync(0xffffffffu, r, 0) != 0;
                }
                tc_wait_ld(x);
                if (!ok) break;
                float* dst = t_buf + (size_t)(c * t_slots + (q % t_slots)) * (32 * kFzTStride) + lane;
#pragma unroll
                for (int j = 0; j < 32; ++j) dst[j * kFzTStride] = __uint_as_float(x[j]);
                __syncwarp();
                if (lane == 0) mbar_arrive(smem_u32(&bars.t_full[c][q]));
            }
            tc_fence_before();
            __syncwarp();
            if (lane == 0 && ok) {
                if (PAIR) mbar_arrive_in(smem_u32(&bars.acc_empty[a]), 0);
                else mbar_arrive(smem_u32(&bars.acc_empty[a]));
            }
        }
    } else {
        // ===== scanner warps: thread = feature row ======================================================
        constexpr float kLog2e = 1.4426950408889634f;
        const int c = warp - (2 + kFzWriterWarps);  // this warp's group of 32 rows
        const int r_local = c * 32 + lane;
        const bool row_ok = r_local < rows;
        if (c < n_chunks) {
            float m_run = -INFINITY, s_run = 0.f;  // running maximum and sum of exp(x - maximum)
            unsigned long long list[kFzMaxK];       // the row's best keys so far, descending
#pragma unroll
            for (int j = 0; j < kFzMaxK; ++j) list[j] = 0ull;
            // Value of the k-th best once k keys are held.  Entries come in ascending token order, so one
            // that only equals it loses the tie: nothing at or below the bar can enter.
            float bar_f = -INFINITY;
            bool ok = true;
            for (int i = 0; i < my_tiles && ok; ++i) {
                const int v0 = (unit + i * units) * tile_v + (int)rank * kFzTileV;
#pragma unroll 1
                for (int q = 0; q < 4 && ok; ++q) {
                    const int c0 = q * 32;
                    int r = 1;
                    if (lane == 0) r = mbar_wait(smem_u32(&bars.t_full[c][q]), (uint32_t)(i & 1), ctl) ? 1 : 0;
                    ok = __shfl_sync(0xffffffffu, r, 0) != 0;
                    __syncwarp();
                    if (!ok) break;
                    const float* src = t_buf + (size_t)(c * t_slots + (q % t_slots)) * (32 * kFzTStride) + lane * kFzTStride;
                    float x[32];
#pragma unroll
                    for (int e = 0; e < 32; ++e) x[e] = src[e];
                    __syncwarp();
                    if (lane == 0) mbar_arrive(smem_u32(&bars.t_empty[c][q]));  // the unit is in registers
                    const int n_valid = V - (v0 + c0);  // vocabulary entries of this unit that exist
                    if (n_valid <= 0) continue;         // (uniform over the block; the units are still taken)
                    if (n_valid < 32) {
#pragma unroll
                        for (int e = 0; e < 32; ++e)
                            if (e >= n_valid) x[e] = -INFINITY;
                    }
                    float cm0 = -INFINITY, cm1 = -INFINITY;
#pragma unroll
                    for (int e = 0; e < 32; e += 2) cm0 = fmaxf(cm0, x[e]), cm1 = fmaxf(cm1, x[e + 1]);
                    const float cm = fmaxf(cm0, cm1);
                    if (cm > m_run) {
                        s_run *= ex2((m_run - cm) * kLog2e);  // 0 when nothing was summed yet
                        m_run = cm;
                    }
                    {   // a NaN or +inf logit leaves a NaN here; -inf adds nothing
                        float acc0 = 0.f, acc1 = 0.f;
                        const float nm = m_run > -INFINITY ? -m_run * kLog2e : 0.f;
#pragma unroll
                        for (int e = 0; e < 32; e += 2) {
                            acc0 += ex2(fmaf(x[e], kLog2e, nm));
                            acc1 += ex2(fmaf(x[e + 1], kLog2e, nm));
                        }
                        s_run += acc0 + acc1;
                    }
                    // Entries that may enter the list (rare once it has settled): a bit per entry, then one
                    // entry per lane and turn of a warp-wide loop, picked out of the registers by a select
                    // tree (indexing them by a run-time value would put the whole chunk into local memory).
                    uint32_t cand = 0u;
                    if (row_ok && cm > bar_f) {
#pragma unroll
                        for (int e = 0; e < 32; ++e)
                            if (x[e] > bar_f) cand |= 1u << e;
                    }
                    while (__any_sync(0xffffffffu, cand != 0u)) {
                        if (cand) {
                            const int e = __ffs(cand) - 1;
                            cand &= cand - 1u;
                            float y16[16], y8[8], y4[4], y2[2];
#pragma unroll
                            for (int j = 0; j < 16; ++j) y16[j] = (e & 16) ? x[16 + j] : x[j];
#pragma unroll
                            for (int j = 0; j < 8; ++j) y8[j] = (e & 8) ? y16[8 + j] : y16[j];
#pragma unroll
                            for (int j = 0; j < 4; ++j) y4[j] = (e & 4) ? y8[4 + j] : y8[j];
#pragma unroll
                            for (int j = 0; j < 2; ++j) y2[j] = (e & 2) ? y4[2 + j] : y4[j];
                            const float f = (e & 1) ? y2[1] : y2[0];
                            if (f > bar_f) {  // the bar may have risen since the bits were set
                                const unsigned long long kth = fz_insert(list, make_key(f, (uint32_t)(v0 + c0 + e)), k);
                                if (kth) bar_f = key_value(kth);
                            }
                        }
                    }
                }
            }
            if (ok && row_ok) {
                const size_t part = (size_t)(row0 + r_local) * slots + blockIdx.x;
                stats[part] = make_double2((double)m_run, (double)s_run);
#pragma unroll
                for (int j = 0; j < kFzMaxK; ++j)
                    if (j < k) keys[part * k + j] = list[j];
                if (!(m_run < INFINITY) || s_run != s_run) raise_status(d_status, EAGLE2_STATUS_NONFINITE_LOGIT);
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

// Units of a launch: blocks (pairs) that walk vocabulary tiles, one per SM (TPC) or fewer when the
// vocabulary has fewer tiles.  Every block writes one partial per row.
static int fz_units(int V, bool pair) {
    const int tile_v = pair ? 2 * kFzTileV : kFzTileV;
    const int n_tiles = (V + tile_v - 1) / tile_v;
    int units = pair ? sm_count() / 2 : sm_count();
    if (units > (pair ? 80 : 160)) units = pair ? 80 : 160;  // never more partials than the row merge holds
    if (units < 1) units = 1;
    return n_tiles < units ? n_tiles : units;
}

// Passes over the weights: all rows in one pass of single blocks up to 128 rows; otherwise passes of
// block pairs with 256 rows each, and the rest in a pass of its own (single blocks up to 128 rows).
struct FzPasses {
    int full;        // pair passes of 256 rows
    int rest;        // rows of the last pass (0: none)
    bool rest_pair;  // the last pass uses block pairs
    int units_pair, units_single;
    int producers_pair, producers_single;  // blocks = partials per row of such a pass
    int slots;                             // partial places per row: the larger of those in use
};
static FzPasses fz_passes(long long rows, int V) {
    FzPasses p;
    p.full = rows > 128 ? (int)(rows / kFzMaxRows) : 0;
    p.rest = (int)(rows - (long long)p.full * kFzMaxRows);
    p.rest_pair = p.rest > 128;
    p.units_pair = fz_units(V, true), p.units_single = fz_units(V, false);
    p.producers_pair = 2 * p.units_pair, p.producers_single = p.units_single;
    const bool any_pair = p.full > 0 || (p.rest && p.rest_pair), any_single = p.rest && !p.rest_pair;
    p.slots = 0;
    if (any_pair) p.slots = p.producers_pair;
    if (any_single && p.producers_single > p.slots) p.slots = p.producers_single;
    if (p.slots < 1) p.slots = 1;
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

// One pass: `rows` feature rows starting at row0 of the call's `rows_total`.
template <bool PAIR>
static int fz_launch(const CUtensorMap& w_map, const void* hidden, long long rows_total, int rows, int row0, int H, int V,
                     int k, int units, int slots, double2* stats, unsigned long long* keys, int32_t* d_status,
                     cudaStream_t st) {
    const int n_pad = (rows + 15) / 16 * 16;       // N of the instruction
    const int b_rows = PAIR ? n_pad / 2 : n_pad;   // feature rows a block copies: a multiple of 8
    const uint32_t b_bytes = (uint32_t)b_rows * kFzTileK * 2;
    const uint32_t stage_bytes = kFzABytes + b_bytes;
    CUtensorMap h_map;
    if (!fz_matrix_map(&h_map, hidden, rows_total, H, b_rows)) return EAGLE2_ERR_CUDA;
    // As many stages as fit beside the transposition units: two per scanner warp with work if that
    // leaves six stages, else one (static shared memory: the barriers).
    cudaFuncAttributes fa;
    if (cudaFuncGetAttributes(&fa, lm_head_topk_kernel<PAIR>) != cudaSuccess) {
        cudaGetLastError();
        return EAGLE2_ERR_CUDA;
    }
    const size_t kDynMax = (size_t)227 * 1024 - fa.sharedSizeBytes;  // what a block may hold, less the static part
    const int n_chunks = (rows + 31) / 32;
    int t_slots = 2;
    int stages = (int)((kDynMax - 1024 - (size_t)n_chunks * t_slots * kFzTBytes) / stage_bytes);
    if (stages < 6) {
        t_slots = 1;
        stages = (int)((kDynMax - 1024 - (size_t)n_chunks * t_slots * kFzTBytes) / stage_bytes);
    }
    if (stages > kFzMaxStages) stages = kFzMaxStages;
    const size_t dyn = 1024 + (size_t)stages * stage_bytes + (size_t)n_chunks * t_slots * kFzTBytes;
    if (cudaFuncSetAttribute(lm_head_topk_kernel<PAIR>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)dyn) != cudaSuccess) {
        cudaGetLastError();
        return EAGLE2_ERR_CUDA;
    }
    return launch_chained(lm_head_topk_kernel<PAIR>, dim3((unsigned)(units * (PAIR ? 2 : 1))), dim3(kFzThreads), dyn, st,
                          PAIR ? 2u : 1u, w_map, h_map, rows, n_pad, row0, H, V, k, stages, t_slots, units, slots, b_bytes,
                          wait_limit_cycles(), stats, keys, d_status);
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
    CUtensorMap w_map;  // vocabulary rows past V read as zero
    if (!fz_matrix_map(&w_map, weight, V, H, kFzTileV)) return EAGLE2_ERR_CUDA;
    cudaStream_t st = reinterpret_cast<cudaStream_t>(stream);
    int rc = EAGLE2_OK;
    for (int i = 0; i < p.full && rc == EAGLE2_OK; ++i)
        rc = fz_launch<true>(w_map, hidden, rows, kFzMaxRows, i * kFzMaxRows, H, V, k, p.units_pair, p.slots, stats, keys,
                             d_status, st);
    if (rc == EAGLE2_OK && p.rest)
        rc = p.rest_pair ? fz_launch<true>(w_map, hidden, rows, p.rest, p.full * kFzMaxRows, H, V, k, p.units_pair, p.slots,
                                           stats, keys, d_status, st)
                         : fz_launch<false>(w_map, hidden, rows, p.rest, p.full * kFzMaxRows, H, V, k, p.units_single, p.slots,
                                            stats, keys, d_status, st);
    if (rc != EAGLE2_OK) return rc;
    const int rest_producers = p.rest_pair ? p.producers_pair : p.producers_single;
    rc = launch_expand_row_merge(B, n_s, p.slots, (long long)p.full * kFzMaxRows, p.full ? p.producers_pair : rest_producers,
                                 p.rest ? rest_producers : p.producers_pair, k, ws, ws_rows, st);
    if (rc != EAGLE2_OK) return rc;
    return launch_expand_merge(B, V, k, D, s, 1, tree_token, tree_parent, tree_value, frontier, ws_rows, d_status, st);
}
