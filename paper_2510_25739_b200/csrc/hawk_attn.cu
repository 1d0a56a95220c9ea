// hawk_verify_attn: block-causal attention of the K draft queries of every guidance stream against
// the cached keys/values (the target model's parallel verification pass, Sec. 3).
//
// The kernel is bound by reading the KV cache once from HBM.  Each thread block owns one
// (stream, kv head, query-head chunk, key split) item and streams its keys through shared memory:
//   - one producer warp issues TMA tile loads (128-byte swizzle) into a ring of stages guarded by
//     full/empty mbarriers;
//   - four consumer warps each take 16 keys of every 64-key tile, compute Q.K^T and P.V with
//     warp-level bf16 MMAs (queries padded to the 16-row operand; the tensor pipe is only an ALU
//     offload here) and keep a running max/sum softmax in registers with quad shuffles;
//   - the four partial results are merged through shared memory and either written as bf16 or, when
//     the keys of an item are split over several blocks, stored as fp32 partials that a small
//     second kernel merges.
#include <math_constants.h>

#include "hawk_common.cuh"

namespace {

using namespace hawk;

constexpr int kConsumerWarps = 4;
constexpr int kKeysPerWarp = 16;
constexpr int kTileKeys = kConsumerWarps * kKeysPerWarp;  // 64 keys per stage
constexpr int kThreads = (kConsumerWarps + 1) * 32;

template <int D>
struct AttnCfg {
    static constexpr int kHalves = D / 64;                        // 64-column (128-byte) sub-tiles
    static constexpr int kSubTileBytes = kTileKeys * 128;         // one [64 keys][64 cols] sub-tile
    static constexpr int kStageBytes = 2 * kHalves * kSubTileBytes;  // K and V
    static constexpr int kStages = D == 64 ? 4 : 3;
    static constexpr int kMergeFloats = kConsumerWarps * 16 * (D + 2);  // aliases the stage ring after the loop
    static_assert(kMergeFloats * sizeof(float) <= static_cast<size_t>(kStages) * kStageBytes, "merge must fit");
    static constexpr size_t kSmemBytes =
        1024 /*align slack*/ + static_cast<size_t>(kStages) * kStageBytes + 2 * kStages * sizeof(uint64_t) + 64;
};

struct AttnParams {
    const __nv_bfloat16 *q;
    const int32_t *prefix_len;
    __nv_bfloat16 *out;
    float *part_o;   // [S][H][K][nsplit][D]
    float *part_ml;  // [S][H][K][nsplit][2]
    int S, K, H, H_kv, L_cap;
    int chunk_heads;  // query heads handled per item (rows = chunk_heads * K <= 16)
    int chunks;       // items per kv head
    int nsplit;
    float scale_log2;  // sm_scale * log2(e)
    int32_t *dev_status;
};

template <int D>
__global__ void __launch_bounds__(kThreads) attn_kernel(const __grid_constant__ CUtensorMap map_k,
                                                        const __grid_constant__ CUtensorMap map_v,
                                                        const AttnParams P)
{
    using C = AttnCfg<D>;
    extern __shared__ uint8_t smem_raw[];
    uint8_t *smem = reinterpret_cast<uint8_t *>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
    uint8_t *stage_base = smem;
    float *merge = reinterpret_cast<float *>(smem);  // reused once every tile has been consumed
    uint64_t *full_bar = reinterpret_cast<uint64_t *>(smem + C::kStages * C::kStageBytes);
    uint64_t *empty_bar = full_bar + C::kStages;
    volatile int *abort_flag = reinterpret_cast<volatile int *>(empty_bar + C::kStages);

    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;

    // ---- which item
    int item = blockIdx.x;
    const int sp = item % P.nsplit;
    item /= P.nsplit;
    const int chunk = item % P.chunks;
    item /= P.chunks;
    const int hk = item % P.H_kv;
    const int s = item / P.H_kv;
    const int group = P.H / P.H_kv;
    const int h0 = hk * group + chunk * P.chunk_heads;                       // first query head of the item
    const int nheads = min(P.chunk_heads, group - chunk * P.chunk_heads);    // heads in this chunk
    const int nrows = nheads * P.K;

    int pl = P.prefix_len[s];
    if (pl < 0 || pl > P.L_cap - P.K) {
        if (tid == 0 && P.dev_status) atomicOr(P.dev_status, HAWK_DEV_BAD_PREFIX);
        pl = max(0, min(pl, P.L_cap - P.K));
    }
    const int n_total = pl + P.K;  // keys any query of this stream can see
    const int tiles = (n_total + kTileKeys - 1) / kTileKeys;
    const int tiles_per_split = (tiles + P.nsplit - 1) / P.nsplit;
    const int t_begin = sp * tiles_per_split;
    const int t_end = min(tiles, t_begin + tiles_per_split);
    const int row_base = (s * P.H_kv + hk) * P.L_cap;  // first cache row of this (stream, kv head)

    if (tid == 0) {
        for (int i = 0; i < C::kStages; ++i) {
            mbar_init(&full_bar[i], 1);
            mbar_init(&empty_bar[i], kConsumerWarps);
        }
        *abort_flag = 0;
        fence_mbar_init();
    }
    __syncthreads();

    if (warp == kConsumerWarps) {
        // =========================== producer warp: one lane issues every tile load
        if (lane == 0) {
            prefetch_tensormap(&map_k);
            prefetch_tensormap(&map_v);
            const uint64_t policy = l2_policy_evict_first();
            int st = 0;
            uint32_t ph = 0;
            bool ok = true;
            int issued = 0;
            uint32_t armed_parity[C::kStages];
            for (int t = t_begin; t < t_end && ok; ++t) {
                if (issued >= C::kStages) ok = mbar_wait(&empty_bar[st], ph ^ 1u, abort_flag);
                if (!ok) break;
                uint8_t *kd = stage_base + st * C::kStageBytes;
                uint8_t *vd = kd + C::kHalves * C::kSubTileBytes;
                mbar_arrive_expect_tx(&full_bar[st], C::kStageBytes);
                armed_parity[st] = ph;
                const int y = row_base + t * kTileKeys;
#pragma unroll
                for (int hf = 0; hf < C::kHalves; ++hf) {
                    tma_load_2d_hint(kd + hf * C::kSubTileBytes, &map_k, hf * 64, y, &full_bar[st], policy);
                    tma_load_2d_hint(vd + hf * C::kSubTileBytes, &map_v, hf * 64, y, &full_bar[st], policy);
                }
                ++issued;
                if (++st == C::kStages) {
                    st = 0;
                    ph ^= 1u;
                }
            }
            if (!ok) {
                *abort_flag = 1;
                if (P.dev_status) atomicOr(P.dev_status, HAWK_DEV_TIMEOUT);
                // let the copies already issued land (bounded) before the block can retire
                for (int i = 0; i < C::kStages && i < issued; ++i) mbar_wait(&full_bar[i], armed_parity[i], nullptr);
            }
        }
        return;  // consumers only use named barrier 1 from here on
    }

    // =========================== consumer warps
    const int g = lane >> 2, tq = lane & 3;  // fragment row / column-pair index
    // row r of the 16-row query operand: head h0 + r / K, draft position r % K (rows >= nrows are padding)
    const int r0 = g, r1 = g + 8;
    const int i0 = r0 % P.K, i1 = r1 % P.K;
    const bool v0 = r0 < nrows, v1 = r1 < nrows;
    const int lim0 = pl + i0 + 1, lim1 = pl + i1 + 1;  // visible keys: j < lim

    // Q fragments (A operand, 16 x D), straight from global memory
    uint32_t qa[D / 16][4];
    {
        const __nv_bfloat16 *q0 = P.q + ((static_cast<size_t>(s) * P.K + i0) * P.H + (h0 + r0 / P.K)) * D;
        const __nv_bfloat16 *q1 = P.q + ((static_cast<size_t>(s) * P.K + i1) * P.H + (h0 + r1 / P.K)) * D;
#pragma unroll
        for (int kk = 0; kk < D / 16; ++kk) {
            const int d = kk * 16 + 2 * tq;
            qa[kk][0] = v0 ? *reinterpret_cast<const uint32_t *>(q0 + d) : 0u;
            qa[kk][1] = v1 ? *reinterpret_cast<const uint32_t *>(q1 + d) : 0u;
            qa[kk][2] = v0 ? *reinterpret_cast<const uint32_t *>(q0 + d + 8) : 0u;
            qa[kk][3] = v1 ? *reinterpret_cast<const uint32_t *>(q1 + d + 8) : 0u;
        }
    }

    float o[D / 8][4];
#pragma unroll
    for (int c = 0; c < D / 8; ++c) o[c][0] = o[c][1] = o[c][2] = o[c][3] = 0.f;
    float m0 = -CUDART_INF_F, m1 = -CUDART_INF_F, l0 = 0.f, l1 = 0.f;  // running max (log2 units) and sum

    int st = 0;
    uint32_t ph = 0;
    bool ok = true;
    const uint32_t stage_u32 = smem_u32(stage_base);
    // ldmatrix row addressing: lane -> (matrix mi = lane / 8, row lane % 8)
    const int lm_mi = lane >> 3, lm_r = lane & 7;

    for (int t = t_begin; t < t_end; ++t) {
        ok = mbar_wait(&full_bar[st], ph, abort_flag);
        if (!ok) break;
        const uint32_t kbase = stage_u32 + st * C::kStageBytes;
        const uint32_t vbase = kbase + C::kHalves * C::kSubTileBytes;
        const int key0 = t * kTileKeys + warp * kKeysPerWarp;  // first key of this warp's slice

        if (key0 < n_total) {
            // ---- scores S = Q K^T for 16 keys: two 8-key column tiles
            float sc[2][4];
#pragma unroll
            for (int nt = 0; nt < 2; ++nt) sc[nt][0] = sc[nt][1] = sc[nt][2] = sc[nt][3] = 0.f;
#pragma unroll
            for (int kk = 0; kk < D / 16; ++kk) {
                // matrices: (keys 0-7, d lo), (keys 0-7, d hi), (keys 8-15, d lo), (keys 8-15, d hi)
                const int krow = warp * kKeysPerWarp + (lm_mi >> 1) * 8 + lm_r;
                const int chunk16 = kk * 2 + (lm_mi & 1);  // 16-byte column chunk 0 .. D/8-1
                const uint32_t addr = kbase + (chunk16 >> 3) * C::kSubTileBytes + krow * 128 +
                                      (((chunk16 & 7) ^ (krow & 7)) << 4);
                uint32_t kb[4];
                ldmatrix_x4(kb, addr);
                mma_bf16_16816(sc[0], qa[kk], kb[0], kb[1]);
                mma_bf16_16816(sc[1], qa[kk], kb[2], kb[3]);
            }
            // ---- causal mask inside the block (only tiles that reach past the prefix)
            if (key0 + kKeysPerWarp > pl) {
#pragma unroll
                for (int nt = 0; nt < 2; ++nt) {
                    const int j = key0 + nt * 8 + 2 * tq;
                    if (j >= lim0) sc[nt][0] = -CUDART_INF_F;
                    if (j + 1 >= lim0) sc[nt][1] = -CUDART_INF_F;
                    if (j >= lim1) sc[nt][2] = -CUDART_INF_F;
                    if (j + 1 >= lim1) sc[nt][3] = -CUDART_INF_F;
                }
            }
            // ---- running softmax (log2 domain), quad shuffles for the row maximum
            float mx0 = fmaxf(fmaxf(sc[0][0], sc[0][1]), fmaxf(sc[1][0], sc[1][1]));
            float mx1 = fmaxf(fmaxf(sc[0][2], sc[0][3]), fmaxf(sc[1][2], sc[1][3]));
            mx0 = fmaxf(mx0, __shfl_xor_sync(0xffffffffu, mx0, 1));
            mx0 = fmaxf(mx0, __shfl_xor_sync(0xffffffffu, mx0, 2));
            mx1 = fmaxf(mx1, __shfl_xor_sync(0xffffffffu, mx1, 1));
            mx1 = fmaxf(mx1, __shfl_xor_sync(0xffffffffu, mx1, 2));
            const float mn0 = fmaxf(m0, mx0 * P.scale_log2), mn1 = fmaxf(m1, mx1 * P.scale_log2);
            const float mu0 = mn0 == -CUDART_INF_F ? 0.f : mn0, mu1 = mn1 == -CUDART_INF_F ? 0.f : mn1;
            const float a0 = fast_exp2(m0 - mu0), a1 = fast_exp2(m1 - mu1);
            m0 = mn0;
            m1 = mn1;
            float p[2][4];
#pragma unroll
            for (int nt = 0; nt < 2; ++nt) {
                p[nt][0] = fast_exp2(fmaf(sc[nt][0], P.scale_log2, -mu0));
                p[nt][1] = fast_exp2(fmaf(sc[nt][1], P.scale_log2, -mu0));
                p[nt][2] = fast_exp2(fmaf(sc[nt][2], P.scale_log2, -mu1));
                p[nt][3] = fast_exp2(fmaf(sc[nt][3], P.scale_log2, -mu1));
            }
            l0 = l0 * a0 + ((p[0][0] + p[0][1]) + (p[1][0] + p[1][1]));
            l1 = l1 * a1 + ((p[0][2] + p[0][3]) + (p[1][2] + p[1][3]));
#pragma unroll
            for (int c = 0; c < D / 8; ++c) {
                o[c][0] *= a0;
                o[c][1] *= a0;
                o[c][2] *= a1;
                o[c][3] *= a1;
            }
            // P as the A operand of P.V (16 rows x 16 keys)
            uint32_t pa[4];
            pa[0] = pack_bf16(p[0][0], p[0][1]);
            pa[1] = pack_bf16(p[0][2], p[0][3]);
            pa[2] = pack_bf16(p[1][0], p[1][1]);
            pa[3] = pack_bf16(p[1][2], p[1][3]);
            // keys at or past n_total hold whatever the cache holds: zero them so 0 * NaN cannot appear
            const bool ragged = key0 + kKeysPerWarp > n_total;
            const int kleft = n_total - key0;  // valid keys in this slice when ragged
#pragma unroll
            for (int c = 0; c < D / 8; c += 2) {
                // matrices: (keys 0-7, chunk c), (keys 8-15, chunk c), (keys 0-7, chunk c+1), (keys 8-15, chunk c+1)
                const int krow = warp * kKeysPerWarp + (lm_mi & 1) * 8 + lm_r;
                const int chunk16 = c + (lm_mi >> 1);
                const uint32_t addr = vbase + (chunk16 >> 3) * C::kSubTileBytes + krow * 128 +
                                      (((chunk16 & 7) ^ (krow & 7)) << 4);
                uint32_t vb[4];
                ldmatrix_x4_trans(vb, addr);
                if (ragged) {
                    // register 0/2: keys 2tq, 2tq+1; register 1/3: keys 2tq+8, 2tq+9 (low half = first key)
                    const int ka = 2 * tq, kb2 = 2 * tq + 8;
                    const uint32_t ma = (ka < kleft ? 0x0000ffffu : 0u) | (ka + 1 < kleft ? 0xffff0000u : 0u);
                    const uint32_t mb = (kb2 < kleft ? 0x0000ffffu : 0u) | (kb2 + 1 < kleft ? 0xffff0000u : 0u);
                    vb[0] &= ma;
                    vb[2] &= ma;
                    vb[1] &= mb;
                    vb[3] &= mb;
                }
                mma_bf16_16816(o[c], pa, vb[0], vb[1]);
                mma_bf16_16816(o[c + 1], pa, vb[2], vb[3]);
            }
        }
        __syncwarp();
        if (lane == 0) mbar_arrive(&empty_bar[st]);
        if (++st == C::kStages) {
            st = 0;
            ph ^= 1u;
        }
    }
    if (!ok) {
        if (lane == 0) {
            *abort_flag = 1;
            if (P.dev_status) atomicOr(P.dev_status, HAWK_DEV_TIMEOUT);
        }
    }

    // ---- merge the four warps' partial softmax states through shared memory
    l0 += __shfl_xor_sync(0xffffffffu, l0, 1);
    l0 += __shfl_xor_sync(0xffffffffu, l0, 2);
    l1 += __shfl_xor_sync(0xffffffffu, l1, 1);
    l1 += __shfl_xor_sync(0xffffffffu, l1, 2);
    asm volatile("bar.sync 1, %0;" ::"n"(kConsumerWarps * 32) : "memory");  // all slices read: ring is free
    float *mw = merge + warp * 16 * (D + 2);
#pragma unroll
    for (int c = 0; c < D / 8; ++c) {
        const int d = c * 8 + 2 * tq;
        *reinterpret_cast<float2 *>(mw + r0 * (D + 2) + d) = make_float2(o[c][0], o[c][1]);
        *reinterpret_cast<float2 *>(mw + r1 * (D + 2) + d) = make_float2(o[c][2], o[c][3]);
    }
    if (tq == 0) {
        mw[r0 * (D + 2) + D] = m0;
        mw[r0 * (D + 2) + D + 1] = l0;
        mw[r1 * (D + 2) + D] = m1;
        mw[r1 * (D + 2) + D + 1] = l1;
    }
    asm volatile("bar.sync 1, %0;" ::"n"(kConsumerWarps * 32) : "memory");

    // every consumer thread finishes a strided set of (row, column pair) outputs
    constexpr int kPairs = D / 2;
    for (int idx = tid; idx < nrows * kPairs; idx += kConsumerWarps * 32) {
        const int r = idx / kPairs, d = (idx - r * kPairs) * 2;
        float mm = -CUDART_INF_F;
#pragma unroll
        for (int w = 0; w < kConsumerWarps; ++w) mm = fmaxf(mm, merge[(w * 16 + r) * (D + 2) + D]);
        const float mu = mm == -CUDART_INF_F ? 0.f : mm;
        float ll = 0.f, ox = 0.f, oy = 0.f;
#pragma unroll
        for (int w = 0; w < kConsumerWarps; ++w) {
            const float *rw = merge + (w * 16 + r) * (D + 2);
            const float f = fast_exp2(rw[D] - mu);
            ll += rw[D + 1] * f;
            const float2 ov = *reinterpret_cast<const float2 *>(rw + d);
            ox += ov.x * f;
            oy += ov.y * f;
        }
        const int h = h0 + r / P.K, i = r % P.K;
        if (P.nsplit == 1) {
            const float inv = 1.f / ll;
            __nv_bfloat162 ob = __floats2bfloat162_rn(ox * inv, oy * inv);
            *reinterpret_cast<__nv_bfloat162 *>(P.out + ((static_cast<size_t>(s) * P.K + i) * P.H + h) * D + d) = ob;
        } else {
            const size_t prow = ((static_cast<size_t>(s) * P.H + h) * P.K + i) * P.nsplit + sp;
            *reinterpret_cast<float2 *>(P.part_o + prow * D + d) = make_float2(ox, oy);
            if (d == 0) *reinterpret_cast<float2 *>(P.part_ml + prow * 2) = make_float2(mm, ll);
        }
    }
}

// Merges the per-split partial results: one warp per (stream, head, draft position) row.
template <int D>
__global__ void attn_combine_kernel(const float *part_o, const float *part_ml, __nv_bfloat16 *out, int rows_total,
                                    int K, int H, int nsplit)
{
    const int row = (blockIdx.x * blockDim.x + threadIdx.x) >> 5;  // (s*H + h)*K + i
    const int lane = threadIdx.x & 31;
    if (row >= rows_total) return;
    float mm = -CUDART_INF_F;
    for (int sp = 0; sp < nsplit; ++sp) mm = fmaxf(mm, part_ml[(static_cast<size_t>(row) * nsplit + sp) * 2]);
    const float mu = mm == -CUDART_INF_F ? 0.f : mm;
    constexpr int PER = D / 32;
    float acc[PER];
#pragma unroll
    for (int c = 0; c < PER; ++c) acc[c] = 0.f;
    float ll = 0.f;
    for (int sp = 0; sp < nsplit; ++sp) {
        const size_t pr = static_cast<size_t>(row) * nsplit + sp;
        const float f = fast_exp2(part_ml[pr * 2] - mu);
        ll += part_ml[pr * 2 + 1] * f;
        if (PER == 2) {
            const float2 v = *reinterpret_cast<const float2 *>(part_o + pr * D + lane * 2);
            acc[0] += v.x * f;
            acc[1] += v.y * f;
        } else {
            const float4 v = *reinterpret_cast<const float4 *>(part_o + pr * D + lane * 4);
            acc[0] += v.x * f;
            acc[1] += v.y * f;
            acc[2] += v.z * f;
            acc[3] += v.w * f;
        }
    }
    const float inv = 1.f / ll;
    const int i = row % K, sh = row / K, h = sh % H, s = sh / H;
    __nv_bfloat16 *dst = out + ((static_cast<size_t>(s) * K + i) * H + h) * D + lane * PER;
#pragma unroll
    for (int c = 0; c < PER; c += 2)
        *reinterpret_cast<__nv_bfloat162 *>(dst + c) = __floats2bfloat162_rn(acc[c] * inv, acc[c + 1] * inv);
}

struct AttnPlan {
    int chunk_heads, chunks, nsplit, items;
};

// Launch shape from host-known sizes only, so that the workspace query and the launch agree.
AttnPlan make_plan(int S, int K, int H, int H_kv, int D, int max_prefix_len, int sm_count)
{
    AttnPlan pl;
    const int group = H / H_kv;
    pl.chunk_heads = group < 16 / K ? group : 16 / K;
    if (pl.chunk_heads < 1) pl.chunk_heads = 1;
    pl.chunks = (group + pl.chunk_heads - 1) / pl.chunk_heads;
    pl.items = S * H_kv * pl.chunks;
    const int tiles = (max_prefix_len + K + kTileKeys - 1) / kTileKeys;
    const int resident = sm_count * (D == 64 ? 3 : 2);  // blocks the GPU holds at once
    int ns = (2 * resident + pl.items - 1) / pl.items;  // aim at two resident sets of blocks
    const int max_by_len = tiles / 4 > 1 ? tiles / 4 : 1;  // at least four tiles per split
    if (ns > max_by_len) ns = max_by_len;
    if (ns < 1) ns = 1;
    if (ns > 64) ns = 64;
    pl.nsplit = ns;
    return pl;
}

}  // namespace

extern "C" size_t hawk_verify_attn_workspace_bytes(int S, int K, int H, int H_kv, int D, int max_prefix_len)
{
    if (S <= 0 || K < 1 || K > 16 || H <= 0 || H_kv <= 0 || H % H_kv != 0 || (D != 64 && D != 128) ||
        max_prefix_len < 0)
        return 0;
    const AttnPlan pl = make_plan(S, K, H, H_kv, D, max_prefix_len, 148);
    if (pl.nsplit == 1) return 0;
    return static_cast<size_t>(S) * H * K * pl.nsplit * (D + 2) * sizeof(float);
}

extern "C" hawk_status hawk_verify_attn(const void *q, const void *k_cache, const void *v_cache,
                                        const int32_t *prefix_len, void *out, int S, int K, int H, int H_kv, int D,
                                        int L_cap, int max_prefix_len, float sm_scale, void *workspace,
                                        size_t workspace_bytes, int32_t *dev_status, hawk_stream_t stream)
{
    if (S < 0 || K < 0 || H < 0 || H_kv < 0 || D < 0 || L_cap < 0 || max_prefix_len < 0) return HAWK_ERR_SHAPE;
    if (S == 0) return HAWK_OK;
    if (!q || !k_cache || !v_cache || !prefix_len || !out) return HAWK_ERR_NULL;
    if (K < 1 || K > 16 || (D != 64 && D != 128) || H < 1 || H_kv < 1 || H % H_kv != 0) return HAWK_ERR_UNSUPPORTED;
    if (max_prefix_len + K > L_cap) return HAWK_ERR_SHAPE;
    if (static_cast<long long>(S) * H_kv * L_cap >= (1ll << 31)) return HAWK_ERR_UNSUPPORTED;
    if (!(sm_scale > 0.f) || isinf(sm_scale)) return HAWK_ERR_PARAM;
    if (!hawk_host::aligned16(q) || !hawk_host::aligned16(k_cache) || !hawk_host::aligned16(v_cache) ||
        !hawk_host::aligned16(out))
        return HAWK_ERR_ALIGN;
    int sm_count = 0;
    if (!hawk_host::is_sm100(&sm_count)) return HAWK_ERR_UNSUPPORTED;
    (void)sm_count;  // the plan uses the B200's 148 SMs so that the workspace query needs no device

    const AttnPlan pl = make_plan(S, K, H, H_kv, D, max_prefix_len, 148);
    const size_t need = hawk_verify_attn_workspace_bytes(S, K, H, H_kv, D, max_prefix_len);
    if (need > 0) {
        if (!workspace || workspace_bytes < need) return HAWK_ERR_WORKSPACE;
        if (!hawk_host::aligned16(workspace)) return HAWK_ERR_ALIGN;
    }

    CUtensorMap map_k, map_v;
    const uint64_t rows = static_cast<uint64_t>(S) * H_kv * L_cap;
    if (!hawk_host::encode_bf16_rows_sw128(&map_k, k_cache, rows, D, kTileKeys, true) ||
        !hawk_host::encode_bf16_rows_sw128(&map_v, v_cache, rows, D, kTileKeys, true))
        return HAWK_ERR_CUDA;

    AttnParams P;
    P.q = static_cast<const __nv_bfloat16 *>(q);
    P.prefix_len = prefix_len;
    P.out = static_cast<__nv_bfloat16 *>(out);
    P.part_o = static_cast<float *>(workspace);
    P.part_ml = P.part_o ? P.part_o + static_cast<size_t>(S) * H * K * pl.nsplit * D : nullptr;
    P.S = S;
    P.K = K;
    P.H = H;
    P.H_kv = H_kv;
    P.L_cap = L_cap;
    P.chunk_heads = pl.chunk_heads;
    P.chunks = pl.chunks;
    P.nsplit = pl.nsplit;
    P.scale_log2 = sm_scale * 1.4426950408889634f;
    P.dev_status = dev_status;

    cudaStream_t st = reinterpret_cast<cudaStream_t>(stream);
    const int grid = pl.items * pl.nsplit;
    cudaError_t err;
    if (D == 64) {
        static bool attr_done = false;
        if (!attr_done) {
            if (cudaFuncSetAttribute(attn_kernel<64>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                     static_cast<int>(AttnCfg<64>::kSmemBytes)) != cudaSuccess)
                return HAWK_ERR_CUDA;
            attr_done = true;
        }
        attn_kernel<64><<<grid, kThreads, AttnCfg<64>::kSmemBytes, st>>>(map_k, map_v, P);
    } else {
        static bool attr_done = false;
        if (!attr_done) {
            if (cudaFuncSetAttribute(attn_kernel<128>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                     static_cast<int>(AttnCfg<128>::kSmemBytes)) != cudaSuccess)
                return HAWK_ERR_CUDA;
            attr_done = true;
        }
        attn_kernel<128><<<grid, kThreads, AttnCfg<128>::kSmemBytes, st>>>(map_k, map_v, P);
    }
    err = cudaGetLastError();
    if (err != cudaSuccess) return HAWK_ERR_CUDA;
    if (pl.nsplit > 1) {
        const int rows_total = S * H * K;
        const int threads = 256, blocks = (rows_total * 32 + threads - 1) / threads;
        if (D == 64)
            attn_combine_kernel<64><<<blocks, threads, 0, st>>>(P.part_o, P.part_ml, P.out, rows_total, K, H, pl.nsplit);
        else
            attn_combine_kernel<128><<<blocks, threads, 0, st>>>(P.part_o, P.part_ml, P.out, rows_total, K, H, pl.nsplit);
        if (cudaGetLastError() != cudaSuccess) return HAWK_ERR_CUDA;
    }
    return HAWK_OK;
}
