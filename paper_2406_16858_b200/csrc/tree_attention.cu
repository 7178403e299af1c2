// Step 3 of the hot path: tree-masked attention of the verification pass (paper Section 4.2: each
// draft token sees the committed cache and its own ancestors only).
//
// Split-KV flash decoding.  The m tree tokens of one sequence and the g = Hq/Hkv query heads that
// share a KV head are packed into M = m*g query rows, so each K/V tile read from HBM serves all of
// them.  A block owns (sequence, KV head, row block, KV split): it keeps its query rows in shared
// memory, streams 64-key K/V tiles through a 3-stage cp.async pipeline, computes Q.K^T and P.V on
// the tensor cores (bf16 in, fp32 accumulate) with an online softmax in registers, and writes either
// the final rows (one split) or an unnormalised partial plus (max, sum) that a merge kernel combines.
#include <cuda_bf16.h>
#include <math.h>

#include "common.cuh"

namespace eagle2 {

constexpr int kTileKeys = 64;
constexpr int kStages = 3;
constexpr int kMaxRowsPerBlock = 256;

struct AttnPlan {
    int g, M, n_rb, RB, warps, splits;
    size_t smem;
};

static void attention_plan(int B, int m, int Hq, int Hkv, int d, int max_kv_len, AttnPlan* p) {
    p->g = Hq / Hkv;
    p->M = m * p->g;
    p->n_rb = (p->M + kMaxRowsPerBlock - 1) / kMaxRowsPerBlock;
    const int per = (p->M + p->n_rb - 1) / p->n_rb;
    p->RB = (per + 15) / 16 * 16;
    p->warps = p->RB / 16;
    const long long items = (long long)B * Hkv * p->n_rb;
    const int per_sm = p->warps <= 4 ? 2 : 1;
    const long long target = 148LL * per_sm;
    const int tiles = (max_kv_len + m + kTileKeys - 1) / kTileKeys;
    long long s = target / (items > 0 ? items : 1);
    if (s < 1) s = 1;
    if (s > (tiles + 1) / 2) s = (tiles + 1) / 2;
    if (s < 1) s = 1;
    p->splits = (int)s;
    p->smem = (size_t)p->RB * d * 2 + (size_t)kStages * 2 * kTileKeys * d * 2;
}

struct AttnWs {
    float* o_part;   // [B][Hkv][splits][n_rb*RB][d]
    float2* ml;      // [B][Hkv][splits][n_rb*RB]  (running max in log2 units, running sum)
};

static size_t attention_ws_layout(int B, int Hkv, int d, const AttnPlan& p, void* base, AttnWs* w) {
    if (p.splits == 1) return 0;
    const size_t rows = (size_t)B * Hkv * p.splits * p.n_rb * p.RB;
    // every operation keeps its arrival counters (B ints) at the start of the workspace and leaves
    // them zero; the partials go behind that region so that a shared workspace stays valid
    size_t off = round_up(sizeof(int) * (size_t)B, kWsAlign);
    char* c = static_cast<char*>(base);
    if (w) w->o_part = reinterpret_cast<float*>(c + off);
    off += round_up(rows * d * sizeof(float), kWsAlign);
    if (w) w->ml = reinterpret_cast<float2*>(c + off);
    off += round_up(rows * sizeof(float2), kWsAlign);
    return off;
}

size_t attention_workspace_bytes(int B, int m, int Hq, int Hkv, int d, int max_kv_len) {
    AttnPlan p;
    attention_plan(B, m, Hq, Hkv, d, max_kv_len, &p);
    return attention_ws_layout(B, Hkv, d, p, nullptr, nullptr);
}

// ---- small PTX wrappers --------------------------------------------------------------------------
__device__ __forceinline__ uint32_t smem_u32(const void* p) {
    return (uint32_t)__cvta_generic_to_shared(p);
}
__device__ __forceinline__ void cp_async16(uint32_t dst, const void* src, bool valid) {
    const int n = valid ? 16 : 0;  // 0 source bytes: the 16 destination bytes are zero-filled
    asm volatile("cp.async.cg.shared.global [%0], [%1], 16, %2;\n" ::"r"(dst), "l"(src), "r"(n));
}
__device__ __forceinline__ void cp_async_commit() { asm volatile("cp.async.commit_group;\n" ::); }
template <int N>
__device__ __forceinline__ void cp_async_wait() {
    asm volatile("cp.async.wait_group %0;\n" ::"n"(N));
}
__device__ __forceinline__ void ldmatrix_x4(uint32_t (&r)[4], uint32_t addr) {
    asm volatile("ldmatrix.sync.aligned.m8n8.x4.shared.b16 {%0,%1,%2,%3}, [%4];\n"
                 : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3])
                 : "r"(addr));
}
__device__ __forceinline__ void ldmatrix_x4_trans(uint32_t (&r)[4], uint32_t addr) {
    asm volatile("ldmatrix.sync.aligned.m8n8.x4.trans.shared.b16 {%0,%1,%2,%3}, [%4];\n"
                 : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3])
                 : "r"(addr));
}
__device__ __forceinline__ void mma_bf16(float (&c)[4], const uint32_t (&a)[4], uint32_t b0, uint32_t b1) {
    asm volatile(
        "mma.sync.aligned.m16n8k16.row.col.f32.bf16.bf16.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, "
        "{%0,%1,%2,%3};\n"
        : "+f"(c[0]), "+f"(c[1]), "+f"(c[2]), "+f"(c[3])
        : "r"(a[0]), "r"(a[1]), "r"(a[2]), "r"(a[3]), "r"(b0), "r"(b1));
}
__device__ __forceinline__ uint32_t pack_bf16(float lo, float hi) {
    const __nv_bfloat162 v = __floats2bfloat162_rn(lo, hi);
    return *reinterpret_cast<const uint32_t*>(&v);
}

// Shared-memory tiles are [row][DH] bf16 with the 16-byte chunks of a row XOR-swizzled by the row
// number, so that the 8 rows an ldmatrix touches fall into 8 different bank groups.
template <int DH>
__device__ __forceinline__ uint32_t tile_off(int row, int chunk) {
    return (uint32_t)(row * DH * 2 + ((chunk ^ (row & 7)) << 4));
}

template <int DH>
__global__ void __launch_bounds__(512)
tree_attention_kernel(const __nv_bfloat16* __restrict__ q, const __nv_bfloat16* __restrict__ k_cache,
                      const __nv_bfloat16* __restrict__ v_cache, const int64_t* __restrict__ kv_off,
                      const int32_t* __restrict__ kv_len, const uint64_t* __restrict__ mask_bits, int m,
                      int Hq, int Hkv, AttnPlan plan, float scale_log2, __nv_bfloat16* __restrict__ out,
                      float* __restrict__ lse, AttnWs ws) {
    constexpr int CH = DH / 8;  // 16-byte chunks per row
    extern __shared__ __align__(128) unsigned char smem[];
    __shared__ uint64_t s_mask[EAGLE2_MAX_M * 2];

    const int g = plan.g, M = plan.M, RB = plan.RB, S = plan.splits;
    int bid = blockIdx.x;
    const int split = bid % S;
    bid /= S;
    const int rb = bid % plan.n_rb;
    bid /= plan.n_rb;
    const int hk = bid % Hkv;
    const int b = bid / Hkv;

    const int tid = threadIdx.x, nthreads = blockDim.x;
    const int warp = tid >> 5, lane = tid & 31;
    const int L = kv_len[b];
    const int n_keys = L + m;
    const int W = (m + 63) / 64;
    const int tiles = (n_keys + kTileKeys - 1) / kTileKeys;
    const int per_split = (tiles + S - 1) / S;
    const int t_begin = min(split * per_split, tiles);
    const int t_end = min(t_begin + per_split, tiles);
    const int nt = t_end - t_begin;

    unsigned char* s_q = smem;
    unsigned char* s_kv = smem + (size_t)RB * DH * 2;
    const uint32_t s_q_u32 = smem_u32(s_q);
    const uint32_t s_kv_u32 = smem_u32(s_kv);
    constexpr uint32_t kTileBytes = kTileKeys * DH * 2;

    const int row0 = rb * RB;  // first packed query row of this block
    const __nv_bfloat16* kbase = k_cache + (kv_off[b] * Hkv + hk) * (long long)DH;
    const __nv_bfloat16* vbase = v_cache + (kv_off[b] * Hkv + hk) * (long long)DH;
    const long long kv_row_stride = (long long)Hkv * DH;

    auto load_tile = [&](int t, int stage) {
        const int key0 = (t_begin + t) * kTileKeys;
        const uint32_t kdst = s_kv_u32 + (uint32_t)stage * 2 * kTileBytes;
        const uint32_t vdst = kdst + kTileBytes;
        for (int idx = tid; idx < kTileKeys * CH; idx += nthreads) {
            const int r = idx / CH, c = idx % CH;
            const int key = key0 + r;
            const bool ok = key < n_keys;
            const long long src = (long long)(ok ? key : 0) * kv_row_stride + c * 8;
            cp_async16(kdst + tile_off<DH>(r, c), kbase + src, ok);
            cp_async16(vdst + tile_off<DH>(r, c), vbase + src, ok);
        }
    };

    // ---- prologue: query rows and mask into shared memory, first K/V tiles in flight ------------
    for (int idx = tid; idx < RB * CH; idx += nthreads) {
        const int r = idx / CH, c = idx % CH;
        const int pr = row0 + r;  // packed row = token * g + head-in-group
        const bool ok = pr < M;
        const int tok = ok ? pr / g : 0, gq = ok ? pr % g : 0;
        const __nv_bfloat16* src = q + (((long long)b * m + tok) * Hq + hk * g + gq) * DH + c * 8;
        cp_async16(s_q_u32 + tile_off<DH>(r, c), src, ok);
    }
    cp_async_commit();
    for (int i = tid; i < m * W; i += nthreads) s_mask[i] = mask_bits[(long long)b * m * W + i];
#pragma unroll
    for (int t = 0; t < kStages - 1; ++t) {
        if (t < nt) load_tile(t, t);
        cp_async_commit();
    }

    // per-thread rows: r_lo = 16*warp + lane/4, r_hi = r_lo + 8
    const int qrow_lo = row0 + warp * 16 + (lane >> 2);
    const int tok_lo = min(qrow_lo, M - 1) / g, tok_hi = min(qrow_lo + 8, M - 1) / g;
    float m_run[2] = {-INFINITY, -INFINITY}, l_run[2] = {0.f, 0.f};
    float oacc[DH / 8][4];
#pragma unroll
    for (int n = 0; n < DH / 8; ++n) oacc[n][0] = oacc[n][1] = oacc[n][2] = oacc[n][3] = 0.f;

    for (int it = 0; it < nt; ++it) {
        cp_async_wait<kStages - 2>();
        __syncthreads();
        if (it + kStages - 1 < nt) load_tile(it + kStages - 1, (it + kStages - 1) % kStages);
        cp_async_commit();

        const uint32_t ks = s_kv_u32 + (uint32_t)(it % kStages) * 2 * kTileBytes;
        const uint32_t vs = ks + kTileBytes;
        const int key0 = (t_begin + it) * kTileKeys;
        const bool need_mask = key0 + kTileKeys > L;

#pragma unroll
        for (int half = 0; half < 2; ++half) {  // 32 keys at a time keeps the register count down
            float sacc[4][4];
#pragma unroll
            for (int n = 0; n < 4; ++n) sacc[n][0] = sacc[n][1] = sacc[n][2] = sacc[n][3] = 0.f;
#pragma unroll
            for (int kk = 0; kk < DH / 16; ++kk) {
                uint32_t a[4];
                ldmatrix_x4(a, s_q_u32 + tile_off<DH>(warp * 16 + (lane & 15), kk * 2 + (lane >> 4)));
#pragma unroll
                for (int np = 0; np < 2; ++np) {  // pairs of 8-key blocks
                    uint32_t bfr[4];
                    const int krow = half * 32 + np * 16 + (lane & 7) + ((lane >> 4) << 3);
                    ldmatrix_x4(bfr, ks + tile_off<DH>(krow, kk * 2 + ((lane >> 3) & 1)));
                    mma_bf16(sacc[np * 2 + 0], a, bfr[0], bfr[1]);
                    mma_bf16(sacc[np * 2 + 1], a, bfr[2], bfr[3]);
                }
            }
            // scale, mask, online softmax
            float mx[2] = {-INFINITY, -INFINITY};
#pragma unroll
            for (int n = 0; n < 4; ++n) {
#pragma unroll
                for (int e = 0; e < 4; ++e) {
                    float sv = sacc[n][e] * scale_log2;
                    if (need_mask) {
                        const int key = key0 + half * 32 + n * 8 + (lane & 3) * 2 + (e & 1);
                        bool vis = key < L;
                        if (!vis && key < n_keys) {
                            const int j = key - L;
                            const int tok = (e & 2) ? tok_hi : tok_lo;
                            vis = (s_mask[tok * W + (j >> 6)] >> (j & 63)) & 1ull;
                        }
                        if (!vis) sv = -INFINITY;
                    }
                    sacc[n][e] = sv;
                    mx[e >> 1] = fmaxf(mx[e >> 1], sv);
                }
            }
            float corr[2];
#pragma unroll
            for (int h = 0; h < 2; ++h) {
                mx[h] = fmaxf(mx[h], __shfl_xor_sync(0xffffffffu, mx[h], 1));
                mx[h] = fmaxf(mx[h], __shfl_xor_sync(0xffffffffu, mx[h], 2));
                const float m_new = fmaxf(m_run[h], mx[h]);
                corr[h] = (m_new == -INFINITY) ? 1.f : exp2f(m_run[h] - m_new);
                m_run[h] = m_new;
                l_run[h] *= corr[h];
            }
            const float base_lo = m_run[0] == -INFINITY ? 0.f : m_run[0];
            const float base_hi = m_run[1] == -INFINITY ? 0.f : m_run[1];
            uint32_t pf[2][4];
#pragma unroll
            for (int n = 0; n < 4; ++n) {
                const float p0 = exp2f(sacc[n][0] - base_lo), p1 = exp2f(sacc[n][1] - base_lo);
                const float p2 = exp2f(sacc[n][2] - base_hi), p3 = exp2f(sacc[n][3] - base_hi);
                l_run[0] += p0 + p1;
                l_run[1] += p2 + p3;
                pf[n >> 1][(n & 1) * 2 + 0] = pack_bf16(p0, p1);
                pf[n >> 1][(n & 1) * 2 + 1] = pack_bf16(p2, p3);
            }
#pragma unroll
            for (int n = 0; n < DH / 8; ++n) {
                oacc[n][0] *= corr[0], oacc[n][1] *= corr[0];
                oacc[n][2] *= corr[1], oacc[n][3] *= corr[1];
            }
            // O += P.V over these 32 keys
#pragma unroll
            for (int kk = 0; kk < 2; ++kk) {
#pragma unroll
                for (int np = 0; np < DH / 16; ++np) {
                    uint32_t bfr[4];
                    const int vrow = half * 32 + kk * 16 + (lane & 7) + (((lane >> 3) & 1) << 3);
                    ldmatrix_x4_trans(bfr, vs + tile_off<DH>(vrow, np * 2 + (lane >> 4)));
                    mma_bf16(oacc[np * 2 + 0], pf[kk], bfr[0], bfr[1]);
                    mma_bf16(oacc[np * 2 + 1], pf[kk], bfr[2], bfr[3]);
                }
            }
        }
    }
    cp_async_wait<0>();

    // ---- epilogue ----------------------------------------------------------------------------
#pragma unroll
    for (int h = 0; h < 2; ++h) {
        l_run[h] += __shfl_xor_sync(0xffffffffu, l_run[h], 1);
        l_run[h] += __shfl_xor_sync(0xffffffffu, l_run[h], 2);
    }
#pragma unroll
    for (int h = 0; h < 2; ++h) {
        const int pr = qrow_lo + h * 8;
        if (pr >= M || pr >= row0 + RB) continue;
        if (S == 1) {
            const int tok = pr / g, gq = pr % g, hq = hk * g + gq;
            const float inv = l_run[h] > 0.f ? 1.f / l_run[h] : 0.f;
            __nv_bfloat16* dst = out + (((long long)b * m + tok) * Hq + hq) * DH;
#pragma unroll
            for (int n = 0; n < DH / 8; ++n) {
                const uint32_t v = pack_bf16(oacc[n][2 * h] * inv, oacc[n][2 * h + 1] * inv);
                *reinterpret_cast<uint32_t*>(dst + n * 8 + (lane & 3) * 2) = v;
            }
            if (lse && (lane & 3) == 0)
                lse[((long long)b * Hq + hq) * m + tok] =
                    (m_run[h] + log2f(l_run[h])) * 0.69314718055994531f;
        } else {
            const size_t prow = (((size_t)b * Hkv + hk) * S + split) * ((size_t)plan.n_rb * RB) + (pr);
            float* dst = ws.o_part + prow * DH;
#pragma unroll
            for (int n = 0; n < DH / 8; ++n)
                *reinterpret_cast<float2*>(dst + n * 8 + (lane & 3) * 2) =
                    make_float2(oacc[n][2 * h], oacc[n][2 * h + 1]);
            if ((lane & 3) == 0) ws.ml[prow] = make_float2(m_run[h], l_run[h]);
        }
    }
}

// One warp per output row: combine the splits' partials.
template <int DH>
__global__ void __launch_bounds__(256)
tree_attention_merge_kernel(int B, int m, int Hq, int Hkv, AttnPlan plan, AttnWs ws,
                            __nv_bfloat16* __restrict__ out, float* __restrict__ lse) {
    const int warp_global = (blockIdx.x * blockDim.x + threadIdx.x) >> 5, lane = threadIdx.x & 31;
    const int g = plan.g, S = plan.splits;
    const long long total = (long long)B * Hkv * plan.M;
    if (warp_global >= total) return;
    const int pr = warp_global % plan.M;
    const int hk = (warp_global / plan.M) % Hkv;
    const int b = warp_global / (plan.M * Hkv);
    const size_t rows_per_split = (size_t)plan.n_rb * plan.RB;
    const size_t first = (((size_t)b * Hkv + hk) * S) * rows_per_split + pr;
    float mmax = -INFINITY;
    for (int s = 0; s < S; ++s) mmax = fmaxf(mmax, ws.ml[first + s * rows_per_split].x);
    constexpr int PER = DH / 32;
    float acc[PER];
#pragma unroll
    for (int e = 0; e < PER; ++e) acc[e] = 0.f;
    float l = 0.f;
    for (int s = 0; s < S; ++s) {
        const float2 ml = ws.ml[first + s * rows_per_split];
        if (ml.x == -INFINITY) continue;
        const float w = exp2f(ml.x - mmax);
        l += ml.y * w;
        const float* src = ws.o_part + (first + s * rows_per_split) * DH + lane * PER;
#pragma unroll
        for (int e = 0; e < PER; ++e) acc[e] += src[e] * w;
    }
    const float inv = l > 0.f ? 1.f / l : 0.f;
    const int tok = pr / g, hq = hk * g + pr % g;
    __nv_bfloat16* dst = out + (((long long)b * m + tok) * Hq + hq) * DH + lane * PER;
#pragma unroll
    for (int e = 0; e < PER; e += 2)
        *reinterpret_cast<uint32_t*>(dst + e) = pack_bf16(acc[e] * inv, acc[e + 1] * inv);
    if (lse && lane == 0)
        lse[((long long)b * Hq + hq) * m + tok] = (mmax + log2f(l)) * 0.69314718055994531f;
}

template <int DH>
static int launch_attention(const void* q, const void* k_cache, const void* v_cache, const int64_t* kv_off,
                            const int32_t* kv_len, const uint64_t* mask_bits, int B, int m, int Hq, int Hkv,
                            const AttnPlan& plan, float scale, void* out, float* lse, const AttnWs& ws,
                            cudaStream_t st) {
    auto kern = tree_attention_kernel<DH>;
    if (cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)plan.smem) !=
        cudaSuccess)
        return EAGLE2_ERR_CUDA;
    const long long blocks = (long long)B * Hkv * plan.n_rb * plan.splits;
    if (blocks > 0x7fffffffLL) return EAGLE2_ERR_SHAPE;
    kern<<<(unsigned)blocks, plan.warps * 32, plan.smem, st>>>(
        static_cast<const __nv_bfloat16*>(q), static_cast<const __nv_bfloat16*>(k_cache),
        static_cast<const __nv_bfloat16*>(v_cache), kv_off, kv_len, mask_bits, m, Hq, Hkv, plan,
        scale * 1.4426950408889634f, static_cast<__nv_bfloat16*>(out), lse, ws);
    if (launch_result() != EAGLE2_OK) return EAGLE2_ERR_CUDA;
    if (plan.splits > 1) {
        const long long warps = (long long)B * Hkv * plan.M;
        const long long mblocks = (warps + 7) / 8;
        if (mblocks > 0x7fffffffLL) return EAGLE2_ERR_SHAPE;
        tree_attention_merge_kernel<DH><<<(unsigned)mblocks, 256, 0, st>>>(
            B, m, Hq, Hkv, plan, ws, static_cast<__nv_bfloat16*>(out), lse);
        return launch_result();
    }
    return EAGLE2_OK;
}

}  // namespace eagle2

using namespace eagle2;

extern "C" int eagle2_tree_attention(const void* q, const void* k_cache, const void* v_cache,
                                     const int64_t* kv_off, const int32_t* kv_len,
                                     const uint64_t* mask_bits, int B, int m, int Hq, int Hkv, int d,
                                     int max_kv_len, float scale, void* out, float* lse, void* ws,
                                     size_t ws_bytes, int32_t* d_status, eagle2_stream_t stream) {
    if (!q || !k_cache || !v_cache || !kv_off || !kv_len || !mask_bits || !out || !d_status)
        return EAGLE2_ERR_NULL;
    if (B < 0 || m < 1 || m > EAGLE2_MAX_M || Hq < 1 || Hkv < 1 || Hq % Hkv || Hq / Hkv > 8 ||
        (d != 64 && d != 128) || max_kv_len < 0)
        return EAGLE2_ERR_SHAPE;
    if (!aligned(q, 16) || !aligned(k_cache, 16) || !aligned(v_cache, 16) || !aligned(out, 16) ||
        !aligned(mask_bits, 8))
        return EAGLE2_ERR_ALIGN;
    if (B == 0) return EAGLE2_OK;
    AttnPlan plan;
    attention_plan(B, m, Hq, Hkv, d, max_kv_len, &plan);
    AttnWs w = {nullptr, nullptr};
    if (plan.splits > 1) {
        if (!ws || !aligned(ws, kWsAlign)) return EAGLE2_ERR_WORKSPACE;
        if (attention_ws_layout(B, Hkv, d, plan, ws, &w) > ws_bytes) return EAGLE2_ERR_WORKSPACE;
    }
    cudaStream_t st = reinterpret_cast<cudaStream_t>(stream);
    if (d == 64)
        return launch_attention<64>(q, k_cache, v_cache, kv_off, kv_len, mask_bits, B, m, Hq, Hkv, plan,
                                    scale, out, lse, w, st);
    return launch_attention<128>(q, k_cache, v_cache, kv_off, kv_len, mask_bits, B, m, Hq, Hkv, plan, scale,
                                 out, lse, w, st);
}
