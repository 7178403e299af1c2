// The LM head fused with the first half of the expansion (paper Section 4.1: the draft model's
// features go through the LM head of the original LLM, and the expansion keeps the k most probable
// tokens of every row).  For many feature rows (rows = sequences x frontier size) the logits are as
// large as the weights, and writing them only to read them back once is most of the step's traffic.
// Here they never leave the SM: a block walks vocabulary tiles, the tensor pipe leaves
// logits[feature row][256 vocabulary entries] in tensor memory, and the epilogue threads - one per
// feature row - fold each tile into the row's running maximum, sum of exponentials and k best
// (value, token) keys.  When a block has walked its tiles it writes one partial per row, in the
// expansion's own workspace layout, and the expansion's merge launch finishes the step from them.
//
// Operand roles are swapped against the plain LM head: the feature rows are the M side of
// tcgen05.mma (128 per instruction, one or two row tiles per pass), a vocabulary tile is its N = 256,
// so that a thread's tensor-memory lane is a feature row and its columns are that row's logits.
//   TMA warp        streams [256 vocabulary rows x 64 hidden columns] weight boxes and the matching
//                   64 columns of the features (from L2) through a ring of stages;
//   MMA warp        one lane issues four K = 16 instructions per stage and row tile;
//   8 epilogue warps read the finished accumulators and update their rows' statistics and keys.
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

constexpr int kFzThreads = 64 + 256;  // TMA warp, MMA warp, eight epilogue warps
constexpr int kFzTileV = 256;         // vocabulary entries per tile = N of the instruction
constexpr int kFzTileK = 64;          // hidden columns per stage (128 bytes, the swizzle span)
constexpr int kFzMaxK = 16;           // keys a row's list holds (children per node the fused path supports)
constexpr int kFzMaxStages = 4;
constexpr uint32_t kFzABytes = 128 * kFzTileK * 2;       // one row tile's share of a stage
constexpr uint32_t kFzBBytes = kFzTileV * kFzTileK * 2;  // the weight box of a stage

struct FzBarriers {
    unsigned long long full[kFzMaxStages], empty[kFzMaxStages];
    unsigned long long acc_full, acc_empty;  // the tile's accumulators are complete / have been read
    unsigned long long drain;
};

__device__ __forceinline__ void fz_tma_2d(uint32_t dst, const CUtensorMap* map, int c0, int c1, uint32_t bar) {
    asm volatile(
        "cp.async.bulk.tensor.2d.shared::cta.global.tile.mbarrier::complete_tx::bytes "
        "[%0], [%1, {%2, %3}], [%4];"
        ::"r"(dst), "l"(map), "r"(c0), "r"(c1), "r"(bar)
        : "memory");
}

// rows: feature rows of this pass (<= 128 * MT); row0: first of them among all rows of the call;
// chunks: partials per row (= blocks of the launch); stats/keys: the expansion's partial arrays.
template <int MT>
__global__ void __launch_bounds__(kFzThreads, 1)
lm_head_topk_kernel(const __grid_constant__ CUtensorMap w_map, const __grid_constant__ CUtensorMap h_map, int rows,
                    int row0, int H, int V, int k, int stages, int chunks, long long wait_limit,
                    double2* __restrict__ stats, unsigned long long* __restrict__ keys, int32_t* d_status) {
    extern __shared__ unsigned char smem_raw[];
    __shared__ FzBarriers bars;
    __shared__ uint32_t s_tmem_base;
    __shared__ WaitCtl s_ctl;
    constexpr uint32_t kStageBytes = MT * kFzABytes + kFzBBytes;
    constexpr uint32_t kTmemCols = MT * kFzTileV;  // 256 or 512

    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    const uint32_t smem_base = (smem_u32(smem_raw) + 1023u) & ~1023u;
    const int n_tiles = (V + kFzTileV - 1) / kFzTileV;
    const int n_kb = H / kFzTileK;
    volatile WaitCtl* ctl = &s_ctl;
    long long issued = 0;  // producer lane: stages requested so far

    if (tid == 0) {
        s_ctl.abort = 0;
        s_ctl.limit = wait_limit;
        for (int s = 0; s < kFzMaxStages; ++s) {
            mbar_init(smem_u32(&bars.full[s]), 1);
            mbar_init(smem_u32(&bars.empty[s]), 1);
        }
        mbar_init(smem_u32(&bars.acc_full), 1);
        mbar_init(smem_u32(&bars.acc_empty), MT * 4);  // one arrival per epilogue warp that has rows
        mbar_init(smem_u32(&bars.drain), 1);
        fence_barrier_init();
    }
    if (warp == 1) {
        tmem_alloc(smem_u32(&s_tmem_base), kTmemCols);
        tmem_relinquish();
    }
    if (warp == 0 && lane == 0) {
        asm volatile("prefetch.tensormap [%0];" ::"l"(&w_map) : "memory");
        asm volatile("prefetch.tensormap [%0];" ::"l"(&h_map) : "memory");
    }
    tc_fence_before();
    __syncthreads();
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
            for (int t = blockIdx.x; t < n_tiles && ok; t += gridDim.x) {
                for (int kb = 0; kb < n_kb; ++kb, ++issued) {
                    if (issued >= stages) ok = mbar_wait_spin(smem_u32(&bars.empty[st]), ph ^ 1u, ctl);
                    if (!ok) break;
                    const uint32_t dst = smem_base + (uint32_t)st * kStageBytes;
                    const uint32_t bar = smem_u32(&bars.full[st]);
                    mbar_expect_tx(bar, kStageBytes);
#pragma unroll
                    for (int mt = 0; mt < MT; ++mt)  // feature rows past the last one read as zero
                        fz_tma_2d(dst + mt * kFzABytes, &h_map, kb * kFzTileK, row0 + mt * 128, bar);
                    fz_tma_2d(dst + MT * kFzABytes, &w_map, kb * kFzTileK, t * kFzTileV, bar);
                    if (++st == stages) st = 0, ph ^= 1u;
                }
            }
        }
    } else if (warp == 1) {
        // ===== MMA issuer: lane 0 alone waits and issues ================================================
        if (lane == 0) {
            constexpr uint32_t idesc = instr_desc(kFzTileV, false, 128);
            const uint64_t d0 = smem_desc(smem_base, 16);
            const uint32_t lo0 = (uint32_t)d0, hi = (uint32_t)(d0 >> 32);
            int i = 0, st = 0;
            uint32_t ph = 0;
            bool ok = true;
            for (int t = blockIdx.x; t < n_tiles && ok; t += gridDim.x, ++i) {
                if (i >= 1) ok = mbar_wait_spin(smem_u32(&bars.acc_empty), (uint32_t)((i - 1) & 1), ctl);
                if (!ok) break;
                tc_fence_after();
                for (int kb = 0; kb < n_kb; ++kb) {
                    ok = mbar_wait_spin(smem_u32(&bars.full[st]), ph, ctl);
                    if (!ok) break;
                    tc_fence_after();
                    const uint32_t a_lo = lo0 + (uint32_t)st * (kStageBytes >> 4);
                    const uint32_t b_lo = a_lo + ((MT * kFzABytes) >> 4);
#pragma unroll
                    for (int mt = 0; mt < MT; ++mt) {
#pragma unroll
                        for (int ks = 0; ks < kFzTileK / 16; ++ks) {
                            const uint32_t ao = ((uint32_t)mt * kFzABytes + (uint32_t)ks * 32u) >> 4, bo = ((uint32_t)ks * 32u) >> 4;
                            if (ks == 0) umma_ss<1, 2>(tmem + mt * kFzTileV, a_lo + ao, hi, b_lo + bo, hi, idesc, kb > 0 ? 1u : 0u);
                            else umma_ss<1, 1>(tmem + mt * kFzTileV, a_lo + ao, hi, b_lo + bo, hi, idesc);
                        }
                    }
                    tc_commit(smem_u32(&bars.empty[st]));
                    if (++st == stages) st = 0, ph ^= 1u;
                }
                if (ok) tc_commit(smem_u32(&bars.acc_full));
            }
        }
    } else {
        // ===== epilogue warps: thread = feature row ====================================================
        // Warp w reads the tensor-memory lanes 32 * (w % 4) .. + 31; warps 2..5 serve row tile 0,
        // warps 6..9 row tile 1.
        constexpr float kLog2e = 1.4426950408889634f;
        const int mt = (warp - 2) >> 2, quad = warp & 3;
        if (mt < MT) {
            const int r_local = mt * 128 + quad * 32 + lane;
            const bool row_ok = r_local < rows;
            const uint32_t t_addr = tmem + ((uint32_t)(quad << 5) << 16) + (uint32_t)mt * kFzTileV;
            float m_run = -INFINITY, s_run = 0.f;  // running maximum and sum of exp(x - maximum)
            unsigned long long list[kFzMaxK];       // the row's best keys so far, descending
#pragma unroll
            for (int j = 0; j < kFzMaxK; ++j) list[j] = 0ull;
            float bar_f = -INFINITY;                // value of the k-th best (no key below it can enter)
            int bad = 0;
            int i = 0;
            bool ok = true;
            for (int t = blockIdx.x; t < n_tiles && ok; t += gridDim.x, ++i) {
                int r = 1;
                if (lane == 0) r = mbar_wait(smem_u32(&bars.acc_full), (uint32_t)(i & 1), ctl) ? 1 : 0;
                ok = __shfl_sync(0xffffffffu, r, 0) != 0;
                if (!ok) break;
                tc_fence_after();
                const int v0 = t * kFzTileV;
                for (int c0 = 0; c0 < kFzTileV; c0 += 32) {
                    uint32_t x[32];
                    tmem_ld32(t_addr + (uint32_t)c0, x);
                    tc_wait_ld(x);
                    const int n_valid = V - (v0 + c0);  // vocabulary entries of this chunk that exist
                    if (n_valid <= 0) break;            // (uniform over the block)
                    float cm = -INFINITY;
#pragma unroll
                    for (int c = 0; c < 32; ++c) {
                        float f = __uint_as_float(x[c]);
                        if (c >= n_valid) f = -INFINITY;
                        x[c] = __float_as_uint(f);
                        bad |= !(f < INFINITY);
                        cm = fmaxf(cm, f);
                    }
                    if (cm > m_run) {
                        s_run *= ex2((m_run - cm) * kLog2e);  // 0 when nothing was summed yet
                        m_run = cm;
                    }
                    if (m_run > -INFINITY) {
                        float acc0 = 0.f, acc1 = 0.f;
                        const float nm = -m_run * kLog2e;
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
                    if (cm >= bar_f && cm > -INFINITY) {
#pragma unroll
                        for (int c = 0; c < 32; ++c) {
                            const float f = __uint_as_float(x[c]);
                            if (f >= bar_f && f > -INFINITY) cand |= 1u << c;
                        }
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
                            const unsigned long long key = make_key(f, (uint32_t)(v0 + c0 + c));
                            if (f >= bar_f) {
                                // insert at its place among the first k entries; the k-th drops out
#pragma unroll
                                for (int j = kFzMaxK - 1; j >= 1; --j) {
                                    if (j < k) {
                                        if (key > list[j - 1]) list[j] = list[j - 1];
                                        else if (key > list[j]) list[j] = key;
                                    }
                                }
                                if (key > list[0]) list[0] = key;
                                unsigned long long kth = 0ull;  // the k-th best's value is the bar once k keys exist
#pragma unroll
                                for (int j = 0; j < kFzMaxK; ++j)
                                    if (j == k - 1) kth = list[j];
                                if (kth) bar_f = key_value(kth);
                            }
                        }
                    }
                }
                tc_fence_before();
                __syncwarp();
                if (lane == 0) mbar_arrive(smem_u32(&bars.acc_empty));
            }
            if (ok && row_ok) {
                const size_t part = (size_t)(row0 + r_local) * chunks + blockIdx.x;
                stats[part] = make_double2((double)m_run, (double)s_run);
#pragma unroll
                for (int j = 0; j < kFzMaxK; ++j)
                    if (j < k) keys[part * k + j] = list[j];
                if (bad) raise_status(d_status, EAGLE2_STATUS_NONFINITE_LOGIT);
            }
        }
    }

    // ---- teardown -----------------------------------------------------------------------------------
    tc_fence_before();
    __syncthreads();
    if (warp == 1) {
        tc_fence_after();
        if (s_ctl.abort) {
            // instructions issued before the wait ran out may still be reading shared memory and
            // writing tensor memory: let them retire (bounded) before either is given back
            if (lane == 0) {
                tc_commit(smem_u32(&bars.drain));
                mbar_drain(smem_u32(&bars.drain), 0);
            }
            __syncwarp();
            tc_fence_after();
        }
        tmem_dealloc(tmem, kTmemCols);
    }
    if (warp == 0 && lane == 0 && s_ctl.abort) {
        // every copy requested for the newest use of each stage must have landed before the block's
        // shared memory is given back
        for (long long j = issued > stages ? issued - stages : 0; j < issued; ++j)
            mbar_drain(smem_u32(&bars.full[j % stages]), (uint32_t)((j / stages) & 1));
    }
    if (tid == 0 && s_ctl.abort) raise_status(d_status, EAGLE2_STATUS_TIMEOUT);
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

// Partials per row: one per block of the launch, one block per SM or per vocabulary tile.
static int fz_chunks(int V) {
    const int n_tiles = (V + kFzTileV - 1) / kFzTileV;
    const int sms = sm_count();
    return n_tiles < sms ? n_tiles : sms;
}

size_t lm_head_expand_workspace_bytes(int B, int V, int k) {
    const size_t a = expand_partials_bytes(B, 1, fz_chunks(V), k), b = expand_partials_bytes(B, k, fz_chunks(V), k);
    return a > b ? a : b;
}

template <int MT>
static int fz_launch(const CUtensorMap& w_map, const CUtensorMap& h_map, int rows, int row0, int H, int V, int k, int chunks,
                     double2* stats, unsigned long long* keys, int32_t* d_status, cudaStream_t st) {
    constexpr uint32_t kStageBytes = MT * kFzABytes + kFzBBytes;
    const int stages = MT == 2 ? 3 : 4;
    const size_t dyn = (size_t)stages * kStageBytes + 1024;
    if (cudaFuncSetAttribute(lm_head_topk_kernel<MT>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)dyn) != cudaSuccess) {
        cudaGetLastError();
        return EAGLE2_ERR_CUDA;
    }
    return launch_chained(lm_head_topk_kernel<MT>, dim3((unsigned)chunks), dim3(kFzThreads), dyn, st, 1, w_map, h_map, rows, row0,
                          H, V, k, stages, chunks, wait_limit_cycles(), stats, keys, d_status);
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
    const int chunks = fz_chunks(V);
    double2* stats = nullptr;
    unsigned long long* keys = nullptr;
    if (!expand_partials_layout(B, n_s, chunks, k, ws, ws_bytes, &stats, &keys)) return EAGLE2_ERR_WORKSPACE;
    CUtensorMap w_map, h_map;
    // vocabulary rows past V and feature rows past the last one read as zero
    if (!fz_matrix_map(&w_map, weight, V, H, kFzTileV) || !fz_matrix_map(&h_map, hidden, rows, H, 128)) return EAGLE2_ERR_CUDA;
    cudaStream_t st = reinterpret_cast<cudaStream_t>(stream);
    // up to 256 feature rows ride on one pass over the weights
    for (long long r0 = 0; r0 < rows; r0 += 256) {
        const int n = (int)(rows - r0 < 256 ? rows - r0 : 256);
        const int rc = n > 128 ? fz_launch<2>(w_map, h_map, n, (int)r0, H, V, k, chunks, stats, keys, d_status, st)
                               : fz_launch<1>(w_map, h_map, n, (int)r0, H, V, k, chunks, stats, keys, d_status, st);
        if (rc != EAGLE2_OK) return rc;
    }
    return launch_expand_merge(B, V, k, D, s, chunks, tree_token, tree_parent, tree_value, frontier, ws, d_status, st);
}
