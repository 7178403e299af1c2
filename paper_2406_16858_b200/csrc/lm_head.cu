// The step in front of the expansion (paper Section 4.1): the draft model's feature of every frontier
// token goes through the LM head of the original LLM, logits[r][v] = sum_h hidden[r][h] * weight[v][h].
//
// With a handful of rows this is a pass over the weight matrix and nothing else: V*H bf16 from HBM,
// a few flops per byte.  It still is a dense contraction, so the arithmetic runs on the tensor path,
// laid out so that the streamed operand fills the instruction: a tile of 128 vocabulary rows is the
// M side of tcgen05.mma, the (padded) feature rows are its N side, and the accumulator in tensor
// memory holds logits[vocabulary row][feature row].  Persistent blocks walk the vocabulary tiles,
// up to four resident per SM: one block's chain of copy, wait and issue sustains about 36 bytes per
// nanosecond, a quarter short of an SM's share of HBM, and several short rings fill the gap better
// than one long ring (measured: 199 us with one block of 8 stages per SM, 160 us with four of 3
// stages, at 10 rows x 4096 x 128256).  A block is warp specialised:
//   TMA warp       streams 128 x 64 weight boxes (and the matching 64 columns of the features, which
//                  stay in L2) through a ring of stages;
//   MMA warp       one thread issues four K = 16 instructions per stage into one of two accumulators;
//   4 store warps  read the finished accumulator (one vocabulary row per thread) and write fp32
//                  logits, coalesced across the 32 vocabulary rows of a warp, while the other
//                  accumulator is being filled.
// Every wait on an mbarrier is bounded: when it runs out the block raises EAGLE2_STATUS_TIMEOUT,
// waits for its own copies in flight, frees its tensor memory and returns.
#include <cuda.h>
#include <cuda_bf16.h>

#include "common.cuh"
#include "tcgen05.cuh"

namespace eagle2 {

constexpr int kLmThreads = 192;  // TMA warp, MMA warp, four store warps
constexpr int kLmTileV = 128;    // vocabulary rows per tile = M of the instruction
constexpr int kLmTileK = 64;     // hidden columns per stage (128 bytes, the swizzle span)
constexpr int kLmMaxRows = 256;  // N of the instruction
constexpr int kLmMaxStages = 8;
constexpr uint32_t kLmWBytes = kLmTileV * kLmTileK * 2;

struct LmBarriers {
    unsigned long long full[kLmMaxStages], empty[kLmMaxStages], acc_full[2], acc_empty[2];
    unsigned long long drain;  // used only after a wait ran out: the block's last instructions have retired
};

__device__ __forceinline__ void tma_load_2d(uint32_t dst, const CUtensorMap* map, int c0, int c1, uint32_t bar) {
    asm volatile(
        "cp.async.bulk.tensor.2d.shared::cta.global.tile.mbarrier::complete_tx::bytes "
        "[%0], [%1, {%2, %3}], [%4];"
        ::"r"(dst), "l"(map), "r"(c0), "r"(c1), "r"(bar)
        : "memory");
}

// n_pad: feature rows rounded up to a multiple of 16 (the instruction's N); acc_cols: accumulator
// stride in tensor-memory columns (>= 32 so that a 32-column read stays inside the allocation);
// tmem_cols: the allocation, a power of two that holds the last 32-column read of either accumulator.
__global__ void __launch_bounds__(kLmThreads, 4)
lm_head_kernel(const __grid_constant__ CUtensorMap w_map, const __grid_constant__ CUtensorMap h_map, int rows,
               int n_pad, int H, int V, int stages, int tmem_cols, long long wait_limit, float* __restrict__ logits,
               int32_t* d_status) {
    extern __shared__ unsigned char smem_raw[];
    __shared__ LmBarriers bars;
    __shared__ uint32_t s_tmem_base;
    __shared__ WaitCtl s_ctl;

    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    const uint32_t smem_base = (smem_u32(smem_raw) + 1023u) & ~1023u;
    const uint32_t h_bytes = (uint32_t)n_pad * kLmTileK * 2;
    const uint32_t stage_bytes = kLmWBytes + h_bytes;
    const int acc_cols = n_pad < 32 ? 32 : n_pad;
    const int n_tiles = (V + kLmTileV - 1) / kLmTileV;
    const int n_kb = H / kLmTileK;
    volatile WaitCtl* ctl = &s_ctl;
    long long issued = 0;  // producer lane: weight stages requested so far

    if (tid == 0) {
        s_ctl.abort = 0;
        s_ctl.limit = wait_limit;
        for (int s = 0; s < kLmMaxStages; ++s) {
            mbar_init(smem_u32(&bars.full[s]), 1);
            mbar_init(smem_u32(&bars.empty[s]), 1);
        }
        for (int a = 0; a < 2; ++a) {
            mbar_init(smem_u32(&bars.acc_full[a]), 1);
            mbar_init(smem_u32(&bars.acc_empty[a]), 4);  // one arrival per store warp
        }
        mbar_init(smem_u32(&bars.drain), 1);
        fence_barrier_init();
    }
    if (warp == 1) {
        tmem_alloc(smem_u32(&s_tmem_base), (uint32_t)tmem_cols);
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
            for (int t = blockIdx.x; t < n_tiles && ok; t += gridDim.x) {
                for (int kb = 0; kb < n_kb; ++kb, ++issued) {
                    const int st = (int)(issued % stages);
                    const uint32_t ph = (uint32_t)((issued / stages) & 1);
                    if (issued >= stages) ok = mbar_wait_spin(smem_u32(&bars.empty[st]), ph ^ 1u, ctl);
                    if (!ok) break;
                    const uint32_t dst = smem_base + (uint32_t)st * stage_bytes;
                    const uint32_t bar = smem_u32(&bars.full[st]);
                    mbar_expect_tx(bar, stage_bytes);
                    tma_load_2d(dst, &w_map, kb * kLmTileK, t * kLmTileV, bar);
                    tma_load_2d(dst + kLmWBytes, &h_map, kb * kLmTileK, 0, bar);
                }
            }
        }
    } else if (warp == 1) {
        // ===== MMA issuer (the warp walks the loop, lane 0 waits and issues) =========================
        const uint32_t idesc = instr_desc(n_pad, false, kLmTileV);
        auto wait_all = [&](uint32_t bar, uint32_t parity) {
            int r = 1;
            if (lane == 0) r = mbar_wait_spin(bar, parity, ctl) ? 1 : 0;
            r = __shfl_sync(0xffffffffu, r, 0);
            return r != 0;
        };
        long long used = 0;
        int i = 0;
        bool ok = true;
        for (int t = blockIdx.x; t < n_tiles && ok; t += gridDim.x, ++i) {
            const int acc = i & 1;
            if (i >= 2) ok = wait_all(smem_u32(&bars.acc_empty[acc]), (uint32_t)(((i >> 1) - 1) & 1));
            if (!ok) break;
            tc_fence_after();
            const uint32_t d_tmem = tmem + (uint32_t)(acc * acc_cols);
            for (int kb = 0; kb < n_kb; ++kb, ++used) {
                const int st = (int)(used % stages);
                ok = wait_all(smem_u32(&bars.full[st]), (uint32_t)((used / stages) & 1));
                if (!ok) break;
                tc_fence_after();
                if (lane == 0) {
                    const uint32_t base = smem_base + (uint32_t)st * stage_bytes;
                    const uint64_t wd0 = smem_desc(base, 16), hd0 = smem_desc(base + kLmWBytes, 16);
#pragma unroll
                    for (int ks = 0; ks < kLmTileK / 16; ++ks)
                        mma_ss(d_tmem, desc_advance(wd0, ks * 32u), desc_advance(hd0, ks * 32u), idesc,
                               (kb | ks) != 0);
                    tc_commit(smem_u32(&bars.empty[st]));
                }
                __syncwarp();
            }
            if (ok && lane == 0) tc_commit(smem_u32(&bars.acc_full[acc]));
            __syncwarp();
        }
    } else {
        // ===== store warps: tensor-memory lanes 32*(warp % 4) .. +31 ================================
        const int quarter = warp & 3;
        int i = 0;
        bool ok = true;
        for (int t = blockIdx.x; t < n_tiles && ok; t += gridDim.x, ++i) {
            const int acc = i & 1;
            int r = 1;
            if (lane == 0) r = mbar_wait(smem_u32(&bars.acc_full[acc]), (uint32_t)((i >> 1) & 1), ctl) ? 1 : 0;
            ok = __shfl_sync(0xffffffffu, r, 0) != 0;
            if (!ok) break;
            tc_fence_after();
            const int v = t * kLmTileV + quarter * 32 + lane;
            const uint32_t taddr = tmem + ((uint32_t)(quarter * 32) << 16) + (uint32_t)(acc * acc_cols);
            for (int c0 = 0; c0 < rows; c0 += 32) {
                uint32_t x[32];
                tmem_ld32(taddr + (uint32_t)c0, x);
                tc_wait_ld(x);
                if (v < V) {
#pragma unroll
                    for (int c = 0; c < 32; ++c)
                        if (c0 + c < rows) logits[(long long)(c0 + c) * V + v] = __uint_as_float(x[c]);
                }
            }
            tc_fence_before();
            __syncwarp();
            if (lane == 0) mbar_arrive(smem_u32(&bars.acc_empty[acc]));
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
        tmem_dealloc(tmem, (uint32_t)tmem_cols);
    }
    if (warp == 0 && lane == 0 && s_ctl.abort) {
        // whoever gave up, and whenever: every copy requested for the newest use of each stage
        // must have landed before the block's shared memory is given back
        for (long long j = issued > stages ? issued - stages : 0; j < issued; ++j)
            mbar_drain(smem_u32(&bars.full[j % stages]), (uint32_t)((j / stages) & 1));
    }
    if (tid == 0 && s_ctl.abort) raise_status(d_status, EAGLE2_STATUS_TIMEOUT);
}

static bool make_matrix_map(CUtensorMap* map, const void* base, long long n_rows, int H, int box_rows) {
    EncodeTiledFn fn = encode_tiled_fn();
    if (!fn) return false;
    const cuuint64_t dims[2] = {(cuuint64_t)H, (cuuint64_t)n_rows};
    const cuuint64_t strides[1] = {(cuuint64_t)H * 2};
    const cuuint32_t box[2] = {(cuuint32_t)kLmTileK, (cuuint32_t)box_rows};
    const cuuint32_t estr[2] = {1, 1};
    return fn(map, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, const_cast<void*>(base), dims, strides, box, estr,
              CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
              CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

}  // namespace eagle2

using namespace eagle2;

// One launch: up to kLmMaxRows feature rows against the whole weight matrix.
static int lm_head_rows(const void* hidden, const void* weight, int rows, int H, int V, float* logits,
                        int32_t* d_status, eagle2_stream_t stream) {
    const int n_pad = (rows + 15) / 16 * 16;
    CUtensorMap w_map, h_map;
    // feature rows past `rows` and vocabulary rows past V read as zero
    if (!make_matrix_map(&w_map, weight, V, H, kLmTileV) || !make_matrix_map(&h_map, hidden, rows, H, n_pad))
        return EAGLE2_ERR_CUDA;
    const uint32_t stage_bytes = kLmWBytes + (uint32_t)n_pad * kLmTileK * 2;
    const int acc_cols = n_pad < 32 ? 32 : n_pad;
    int tmem_cols = 32;
    while (tmem_cols < acc_cols + (rows + 31) / 32 * 32) tmem_cols <<= 1;
    // resident blocks per SM: four with rings of 2-3 stages where shared memory and the 512
    // tensor-memory columns allow (measured best up to 64 rows), else as many as keep 3 stages each,
    // else one block with the longest ring that fits
    constexpr uint32_t kSmemPerSm = 227u * 1024u, kPerBlockOverhead = 2u * 1024u + 512u;
    int resident = 1, stages = 0;
    for (int c = 4; c >= 1; --c) {
        const int s = (int)((kSmemPerSm / c - kPerBlockOverhead) / stage_bytes);
        if ((s >= (c == 4 ? 2 : 3) && c * tmem_cols <= 512) || c == 1) {
            resident = c;
            stages = c == 1 ? (s > kLmMaxStages ? kLmMaxStages : s) : (s < 3 ? s : 3);
            break;
        }
    }
    const size_t dyn = (size_t)stages * stage_bytes + 1024;
    int dev = 0, sms = 0;
    if (cudaGetDevice(&dev) != cudaSuccess ||
        cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess ||
        // always the device's opt-in maximum, whatever this call needs: concurrent callers with
        // different row counts then set the same value
        cudaFuncSetAttribute(lm_head_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)kSmemPerSm - 1024) !=
            cudaSuccess ||
        cudaFuncSetAttribute(lm_head_kernel, cudaFuncAttributePreferredSharedMemoryCarveout,
                             cudaSharedmemCarveoutMaxShared) != cudaSuccess) {
        cudaGetLastError();
        return EAGLE2_ERR_CUDA;
    }
    const int n_tiles = (V + kLmTileV - 1) / kLmTileV;
    const int grid = n_tiles < resident * sms ? n_tiles : resident * sms;
    return launch_chained(lm_head_kernel, dim3(grid), dim3(kLmThreads), dyn, reinterpret_cast<cudaStream_t>(stream), 1,
                          w_map, h_map, rows, n_pad, H, V, stages, tmem_cols, wait_limit_cycles(), logits, d_status);
}

extern "C" int eagle2_lm_head(const void* hidden, const void* weight, int rows, int H, int V, float* logits,
                              int32_t* d_status, eagle2_stream_t stream) {
    if (!hidden || !weight || !logits || !d_status) return EAGLE2_ERR_NULL;
    if (rows < 0 || H < kLmTileK || H % kLmTileK != 0 || V < 1) return EAGLE2_ERR_SHAPE;
    if (!aligned(hidden, 16) || !aligned(weight, 16) || !aligned(logits, 4)) return EAGLE2_ERR_ALIGN;
    // more rows than one instruction's N: one pass over the weights per 256 rows (at that width a
    // pass is bound by the tensor pipe, not by the weight stream, so little is lost by re-reading)
    for (int r0 = 0; r0 < rows; r0 += kLmMaxRows) {
        const int n = rows - r0 < kLmMaxRows ? rows - r0 : kLmMaxRows;
        const int rc = lm_head_rows(static_cast<const __nv_bfloat16*>(hidden) + (size_t)r0 * H, weight, n, H, V,
                                    logits + (size_t)r0 * V, d_status, stream);
        if (rc != EAGLE2_OK) return rc;
    }
    return EAGLE2_OK;
}
