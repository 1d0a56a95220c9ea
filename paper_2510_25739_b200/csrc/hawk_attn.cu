// hawk_verify_attn: block-causal attention of the K draft queries of every guidance stream against
// the cached keys/values (the target model's parallel verification pass, Sec. 3).
//
// The kernel is bound by reading the KV cache once from HBM, so it is organised around keeping
// that stream of bytes flowing without a gap:
//   - The work is the flat list of KV tiles (item-major; an item is one (stream, kv head, chunk of
//     <= 32 query rows), a tile is kTileKeys consecutive keys).  The list is cut into equal contiguous
//     shares, one per warp of a persistent grid (one block per SM), so every warp reads the same
//     number of bytes whatever the shape of the batch and no wave of blocks is ever partly empty.
//   - Each warp is its own pipeline: lane 0 issues TMA tile loads (128-byte swizzle) into the warp's
//     private ring of stages and re-arms a stage right after the warp has consumed it; there is no
//     block-wide synchronisation after start-up.
//   - Per tile the warp computes the transposed products S^T = K.Q^T and O^T = V^T.P^T with warp-level
//     bf16 MMAs: the keys (and the head dimension) sit on the 16-row operand, the handful of draft
//     queries on the 8-column operand, so a block of K <= 8 drafts wastes no tensor work and the
//     per-key softmax work is a quarter of the query-major form.  The tensor pipe is only an ALU
//     offload here; running max/sum softmax stays in registers (one max reduction per tile).
//     Which block rows a query sees is a 32-bit mask per query: the causal rule for a chain of
//     drafts, the ancestor set for a candidate tree (hawk_verify_attn_tree).
//   - A share that holds all tiles of an item writes bf16 output straight from registers.  A share
//     that holds only part of an item stores an fp32 partial (o, max, sum) in the workspace, and a
//     small second kernel merges the partials of every item that was cut.
#include <math_constants.h>

#include <atomic>

#include "hawk_common.cuh"

namespace {

using namespace hawk;

#ifndef HAWK_ATTN_WARPS
#define HAWK_ATTN_WARPS 8
#endif
#ifndef HAWK_ATTN_STAGE_KB
#define HAWK_ATTN_STAGE_KB 8
#endif
// Two launch shapes share one kernel (WARPS independent pipelines per block, STAGES tiles deep each;
// WARPS * STAGES * 8 KB = 192 KB of shared memory either way):
//   shares: 8 warps x 3 stages.  The flat tile list is cut into equal shares, items may be cut.
//   whole : 3 warps x 8 stages.  One warp per item, no item is cut and no merge kernel runs; only a
//           third of the warps work, so each gets a deeper ring to keep as many bytes in flight.
//           Taken when the items fit (at most 3 per SM) and an item is short enough for one warp.
constexpr int kWarpsShares = HAWK_ATTN_WARPS, kStagesShares = 3;
constexpr int kWarpsWhole = 3, kStagesWhole = 8;
constexpr int kWarpsGroup = 4, kStagesGroup = 2;  // blocks of 4 warps, three per SM: an item's 4 warps merge in shared memory
constexpr int kWholeMaxTiles = 12;       // longest item (in tiles) that one warp takes alone: a lone warp needs
                                         // 0.75 us per tile, so beyond this the shares (and their merge) win
constexpr int kStageBytes = HAWK_ATTN_STAGE_KB * 1024;  // K and V tile of one stage
constexpr int kPlanSms = 148;           // launch shape is planned for the B200's 148 SMs

template <int D>
struct AttnCfg {
    static constexpr int kHalves = D / 64;                       // 64-column (128-byte) sub-tiles
    static constexpr int kTileKeys = kStageBytes / (4 * D);      // keys per stage (K row + V row = 4*D bytes)
    static_assert(kTileKeys % 16 == 0 && kTileKeys >= 16, "a tile is a whole number of 16-key MMA blocks");
    static constexpr int kSubTileBytes = kTileKeys * 128;        // one [keys][64 cols] sub-tile
    static_assert(2 * kHalves * kSubTileBytes == kStageBytes, "stage = K tile + V tile");
    static constexpr size_t smem_bytes(int warps, int stages)
    {
        return 1024 /*align slack*/ + static_cast<size_t>(warps) * stages * kStageBytes + warps * stages * sizeof(uint64_t) +
               64 /*one flag per warp: the warp left a partial result in its ring (group mode)*/;
    }
};

struct AttnParams {
    const __nv_bfloat16 *q;
    const int32_t *prefix_len;
    __nv_bfloat16 *out;
    float *part;  // [workers][2 slots]{o[rows_per_item][D], (running max in log2 units, running sum)[rows_per_item]}
    int S, K, H, H_kv, L_cap;
    int pl_max;           // largest admissible prefix length: min(L_cap - K, max_prefix_len)
    const uint64_t *anc_mask;  // [K] block rows visible to each query position; NULL: causal (row i sees rows <= i)
    int rows_per_item;    // query rows per item, a multiple of 8: the (head of the group, position) pairs of one
                          // kv head, numbered head-major, are cut into chunks of this many rows
    int chunks;           // items per kv head
    int tiles_per_item;   // tiles of the longest admissible prefix: ceil((max_prefix_len + K) / kTileKeys)
    int workers;          // warps that own a share of the flat tile list
    long long total_tiles;  // items * tiles_per_item
    int group_g;            // > 0: every item is split evenly over this many warps of one block, merged in shared memory
    int items;              // items in the call
    int idx32;              // (total_tiles + 1) * workers fits 31 bits: the merge kernel may index in 32 bits
    float scale_log2;     // sm_scale * log2(e)
    int32_t *dev_status;
};

// Flat tile f belongs to worker owner(f); worker g owns [share_begin(g), share_begin(g + 1)).
__host__ __device__ __forceinline__ long long share_begin(long long g, long long T, int G) { return g * T / G; }
__host__ __device__ __forceinline__ int owner(long long f, long long T, int G)
{
    return static_cast<int>(((f + 1) * G - 1) / T);
}

// Position in the flat tile list, decoded.
struct Cursor {
    long long f;
    int item, tile;             // tile index inside the item
    int s, hk, chunk;           // stream, kv head, row chunk
    int pl;                     // clamped prefix length of the stream
    int ntiles;                 // tiles that hold visible keys for this stream
    int row_base;               // first cache row of (s, hk)
};

template <int TK>
__device__ __forceinline__ void decode_item(Cursor &c, const AttnParams &P, int &flags)
{
    c.item = static_cast<int>(c.f / P.tiles_per_item);
    c.tile = static_cast<int>(c.f - static_cast<long long>(c.item) * P.tiles_per_item);
    int it = c.item;
    c.chunk = it % P.chunks;
    it /= P.chunks;
    c.hk = it % P.H_kv;
    c.s = it / P.H_kv;
    int pl = P.prefix_len[c.s];
    if (pl < 0 || pl > P.pl_max) {
        flags |= HAWK_DEV_BAD_PREFIX;
        pl = max(0, min(pl, P.pl_max));
    }
    c.pl = pl;
    c.ntiles = (pl + P.K + TK - 1) / TK;
    c.row_base = (c.s * P.H_kv + c.hk) * P.L_cap;
}

// Moves the cursor to the next tile at or after its position that holds visible keys; false when
// the share is exhausted.  Tiles past a stream's last visible key are skipped without a load.
template <int TK>
__device__ __forceinline__ bool seek_valid(Cursor &c, long long f_end, const AttnParams &P, int &flags)
{
    while (c.f < f_end) {
        if (c.tile < c.ntiles) return true;
        c.f += P.tiles_per_item - c.tile;  // first tile of the next item
        if (c.f >= f_end) return false;
        decode_item<TK>(c, P, flags);
    }
    return false;
}

template <int TK>
__device__ __forceinline__ void step(Cursor &c, long long f_end, const AttnParams &P, int &flags)
{
    ++c.f;
    ++c.tile;
    if (c.tile == P.tiles_per_item && c.f < f_end) decode_item<TK>(c, P, flags);
}

// Is the key `rel` rows past the prefix visible to a query whose block-row mask is m?  Prefix keys
// (rel < 0) always are; block rows past the 64th never are.
__device__ __forceinline__ bool key_visible(int rel, uint64_t m)
{
    return rel < 0 || (rel < 64 && ((m >> rel) & 1ull));
}

// Mask of position `pos` of a plain chain: block rows 0 .. pos.
__device__ __forceinline__ uint64_t chain_mask(int pos) { return pos >= 63 ? ~0ull : (2ull << pos) - 1ull; }

__device__ __forceinline__ uint32_t movmatrix_trans(uint32_t x)
{
    uint32_t y;
    asm volatile("movmatrix.sync.aligned.m8n8.trans.b16 %0, %1;" : "=r"(y) : "r"(x));
    return y;
}

// NQT = number of 8-query column tiles of an item: rows_per_item / 8 (1..4 at D = 64, 1..3 at D = 128).
template <int D, int NQT, int kWarps, int kStages>
__global__ void __launch_bounds__(kWarps * 32, kWarps == kWarpsGroup ? 3 : 1) attn_kernel(const __grid_constant__ CUtensorMap map_k,
                                                           const __grid_constant__ CUtensorMap map_v,
                                                           const AttnParams P)
{
    using C = AttnCfg<D>;
    constexpr int TK = C::kTileKeys;
    constexpr int KB = TK / 16;  // 16-key MMA blocks per tile
    constexpr int DB = D / 16;   // 16-wide blocks of the head dimension
    extern __shared__ uint8_t smem_raw[];
    uint8_t *smem = reinterpret_cast<uint8_t *>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
    uint64_t *bars = reinterpret_cast<uint64_t *>(smem + kWarps * kStages * kStageBytes);
    volatile int *has_part = reinterpret_cast<volatile int *>(bars + kWarps * kStages);  // [kWarps], group mode

    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    // No allow_dependent_launch() here: with the merge kernel's blocks resident and waiting from the
    // start, this kernel measured 10 % slower; the merge kernel is released when the blocks exit.
    if (tid == 0) {
        for (int i = 0; i < kWarps * kStages; ++i) mbar_init(&bars[i], 1);
        for (int i = 0; i < kWarps; ++i) has_part[i] = 0;
        fence_mbar_init();
        fence_proxy_async();
    }
    __syncthreads();  // the only block-wide synchronisation: from here on every warp runs alone
    grid_dependency_wait();

    // shares: the warps of a block take neighbouring shares; whole: items are dealt out to the blocks in turn
    const int w = kWarps == kWarpsWhole ? warp * static_cast<int>(gridDim.x) + static_cast<int>(blockIdx.x)
                                        : static_cast<int>(blockIdx.x) * kWarps + warp;
    const bool grouped = kWarps == kWarpsGroup && P.group_g > 0;
    const bool idle = w >= P.workers;
    if (idle && !grouped) return;  // (a grouped block meets again at the end: its idle warps walk an empty share)
    uint8_t *ring = smem + warp * kStages * kStageBytes;
    uint64_t *full_bar = bars + warp * kStages;
    const uint32_t ring_u32 = smem_u32(ring);

    const long long T = P.total_tiles;
    const long long f_begin = idle ? 0 : share_begin(w, T, P.workers), f_end = idle ? 0 : share_begin(w + 1, T, P.workers);
    int flags = 0;

    uint64_t policy = 0;
    if (lane == 0) {
        prefetch_tensormap(&map_k);
        prefetch_tensormap(&map_v);
        policy = l2_policy_evict_first();
    }

    // ---- issue side: runs up to kStages tiles ahead of the consume side
    Cursor ci;
    ci.f = f_begin;
    decode_item<TK>(ci, P, flags);
    auto issue = [&](const Cursor &c, int st) {
        if (lane == 0) {
            uint8_t *kd = ring + st * kStageBytes;
            uint8_t *vd = kd + C::kHalves * C::kSubTileBytes;
            // (test builds only: the first tile of the first share is armed for more bytes than arrive)
            const bool stall = kTestStallBytes != 0 && blockIdx.x == 0 && warp == 0 && c.f == f_begin;
            mbar_arrive_expect_tx(&full_bar[st], kStageBytes + (stall ? kTestStallBytes : 0u));
            const int y = c.row_base + c.tile * TK;
#pragma unroll
            for (int hf = 0; hf < C::kHalves; ++hf) {
                tma_load_2d_hint(kd + hf * C::kSubTileBytes, &map_k, hf * 64, y, &full_bar[st], policy);
                tma_load_2d_hint(vd + hf * C::kSubTileBytes, &map_v, hf * 64, y, &full_bar[st], policy);
            }
        }
    };
    int in_flight = 0;  // stages armed and not yet consumed
#pragma unroll
    for (int i = 0; i < kStages; ++i) {
        if (seek_valid<TK>(ci, f_end, P, flags)) {
            issue(ci, i);
            step<TK>(ci, f_end, P, flags);
            ++in_flight;
        }
    }

    // ---- consume side.  Fragment coordinates of this thread: g = lane / 4, tq = lane % 4.
    //   S^T block (16 keys x 8 queries): keys g and g + 8, queries 2tq and 2tq + 1 of the column tile
    //   O^T block (16 dims x 8 queries): dims g and g + 8,  queries 2tq and 2tq + 1
    const int g = lane >> 2, tq = lane & 3;
    const int lm_mi = lane >> 3, lm_r = lane & 7;  // ldmatrix: this lane addresses row lm_r of matrix lm_mi
    const int group = P.H / P.H_kv;

    // byte offsets inside a stage of the ldmatrix rows this lane addresses (128-byte swizzle: the
    // 16-byte chunk index is XOR-ed with the row index modulo 8)
    //   K (plain):      matrices (keys 0-7, chunk 2kk), (keys 8-15, 2kk), (keys 0-7, 2kk+1), (keys 8-15, 2kk+1)
    //   V (transposed): matrices (keys 0-7, chunk 2db), (keys 0-7, 2db+1), (keys 8-15, 2db), (keys 8-15, 2db+1)
    uint32_t k_off[DB], v_off[DB];
#pragma unroll
    for (int kk = 0; kk < DB; ++kk) {
        const int kc = 2 * kk + (lm_mi >> 1), vc = 2 * kk + (lm_mi & 1);
        k_off[kk] = (kc >> 3) * C::kSubTileBytes + ((lm_mi & 1) * 8 + lm_r) * 128 + (((kc & 7) ^ lm_r) << 4);
        v_off[kk] = (vc >> 3) * C::kSubTileBytes + ((lm_mi >> 1) * 8 + lm_r) * 128 + (((vc & 7) ^ lm_r) << 4);
    }

    uint32_t qb[NQT][DB][2];  // Q^T as the 16 x 8 operand: query row = column tile * 8 + g
    float ot[NQT][DB][4];     // O^T accumulators
    float mrun[NQT][2], lrun[NQT][2];  // running max (log2 units) and this thread's share of the running sum
    int cur_item = -1, hbase = 0, gr0 = 0, nrows = 0, seg_pl = 0, seg_s = 0;
    long long seg_start = 0;

    // Writes the finished segment: final bf16 rows if the share held the whole item, else an fp32 partial.
    auto flush = [&]() {
        if (cur_item < 0) return;
#pragma unroll
        for (int nq = 0; nq < NQT; ++nq)
#pragma unroll
            for (int c = 0; c < 2; ++c) {
                float l = lrun[nq][c];
                l += __shfl_xor_sync(0xffffffffu, l, 4);
                l += __shfl_xor_sync(0xffffffffu, l, 8);
                l += __shfl_xor_sync(0xffffffffu, l, 16);
                lrun[nq][c] = l;
            }
        const long long a = static_cast<long long>(cur_item) * P.tiles_per_item, b = a + P.tiles_per_item;
        const bool complete = a >= f_begin && b <= f_end;
        if (complete) {
#pragma unroll
            for (int nq = 0; nq < NQT; ++nq) {
                const float inv0 = 1.f / lrun[nq][0], inv1 = 1.f / lrun[nq][1];
                const int r = nq * 8 + g;  // after the transposes below this thread holds query row r
                const bool valid = r < nrows;
                __nv_bfloat16 *dst = P.out + ((static_cast<size_t>(seg_s) * P.K + (gr0 + r) % P.K) * P.H +
                                              (hbase + (gr0 + r) / P.K)) * D + 2 * tq;
#pragma unroll
                for (int db = 0; db < DB; ++db) {
                    // (dims g / g+8) x (queries 2tq, 2tq+1)  ->  (query g) x (dims 2tq, 2tq+1 / +8)
                    const uint32_t lo = movmatrix_trans(pack_bf16(ot[nq][db][0] * inv0, ot[nq][db][1] * inv1));
                    const uint32_t hi = movmatrix_trans(pack_bf16(ot[nq][db][2] * inv0, ot[nq][db][3] * inv1));
                    if (valid && HAWK_IN_BOUNDS(P.dev_status, (dst - P.out) + db * 16 + 9,
                                                static_cast<long long>(P.S) * P.K * P.H * D)) {
                        *reinterpret_cast<uint32_t *>(dst + db * 16) = lo;
                        *reinterpret_cast<uint32_t *>(dst + db * 16 + 8) = hi;
                    }
                }
            }
        } else {
            const int slot = seg_start == f_begin ? 0 : 1;
            // grouped: the warp's ring is free by now (every copy issued has been consumed) and takes the partial
            float *ps = grouped ? reinterpret_cast<float *>(ring)
                                : P.part + (static_cast<size_t>(w) * 2 + slot) * P.rows_per_item * (D + 2);
            if (grouped && lane == 0) has_part[warp] = 1;
            // (debug build: a partial must fit the warp's ring, or its slot of the workspace)
            if (!HAWK_IN_BOUNDS(P.dev_status, P.rows_per_item * (D + 2) * 4 - 1,
                                grouped ? kStages * kStageBytes : P.rows_per_item * (D + 2) * 4) ||
                !HAWK_IN_BOUNDS(P.dev_status, grouped ? 0 : w * 2 + slot, grouped ? 1 : P.workers * 2))
                return;
#pragma unroll
            for (int nq = 0; nq < NQT; ++nq)
#pragma unroll
                for (int c = 0; c < 2; ++c) {
                    const int r = nq * 8 + 2 * tq + c;
                    if (r < nrows) {
                        float *pr = ps + r * D;
#pragma unroll
                        for (int db = 0; db < DB; ++db) {
                            pr[db * 16 + g] = ot[nq][db][c];
                            pr[db * 16 + 8 + g] = ot[nq][db][2 + c];
                        }
                        if (g == 0)
                            *reinterpret_cast<float2 *>(ps + P.rows_per_item * D + 2 * r) =
                                make_float2(mrun[nq][c], lrun[nq][c]);
                    }
                }
        }
    };

    // Q^T operand of one item, straight from global memory (rows past the item's last are zero)
    uint32_t qn[NQT][DB][2];  // the same for the item that follows in the share, fetched ahead
    int qn_item = -1;
    auto load_q = [&](uint32_t (&dst)[NQT][DB][2], int item) {
        int it = item;
        const int chunk = it % P.chunks;
        it /= P.chunks;
        const int hk = it % P.H_kv, s = it / P.H_kv;
        const int first = chunk * P.rows_per_item;  // first row of the chunk among the kv head's group * K rows
        const int rows = min(P.rows_per_item, group * P.K - first);
#pragma unroll
        for (int nq = 0; nq < NQT; ++nq) {
            const int r = nq * 8 + g;  // query row whose values this thread feeds into the operand
            const bool valid = r < rows;
            const __nv_bfloat16 *qr = P.q + ((static_cast<size_t>(s) * P.K + (first + r) % P.K) * P.H +
                                             (hk * group + (first + r) / P.K)) * D + 2 * tq;
#pragma unroll
            for (int kk = 0; kk < DB; ++kk) {
                dst[nq][kk][0] = valid ? *reinterpret_cast<const uint32_t *>(qr + kk * 16) : 0u;
                dst[nq][kk][1] = valid ? *reinterpret_cast<const uint32_t *>(qr + kk * 16 + 8) : 0u;
            }
        }
    };

    Cursor cc;
    cc.f = f_begin;
    decode_item<TK>(cc, P, flags);
    int st = 0;
    uint32_t ph = 0;
    bool ok = true;
    while (seek_valid<TK>(cc, f_end, P, flags)) {
        if (cc.item != cur_item) {
            // ---- a new segment: write the previous one, fetch this item's queries, reset the state
            flush();
            cur_item = cc.item;
            seg_start = cc.f;
            seg_pl = cc.pl;
            seg_s = cc.s;
            hbase = cc.hk * group;
            gr0 = cc.chunk * P.rows_per_item;
            nrows = min(P.rows_per_item, group * P.K - gr0);
            if (qn_item == cc.item) {
#pragma unroll
                for (int nq = 0; nq < NQT; ++nq)
#pragma unroll
                    for (int kk = 0; kk < DB; ++kk) {
                        qb[nq][kk][0] = qn[nq][kk][0];
                        qb[nq][kk][1] = qn[nq][kk][1];
                    }
            } else {
                load_q(qb, cc.item);
            }
            // the next item of the share follows in a few tiles: fetch its queries now, off the critical path
            qn_item = cc.item + 1;
            if (static_cast<long long>(qn_item) * P.tiles_per_item < f_end) load_q(qn, qn_item);
            else qn_item = -1;
#pragma unroll
            for (int nq = 0; nq < NQT; ++nq) {
#pragma unroll
                for (int db = 0; db < DB; ++db) ot[nq][db][0] = ot[nq][db][1] = ot[nq][db][2] = ot[nq][db][3] = 0.f;
#pragma unroll
                for (int c = 0; c < 2; ++c) {
                    mrun[nq][c] = -CUDART_INF_F;
                    lrun[nq][c] = 0.f;
                }
            }
        }
        const int pl = seg_pl;
        const int n_total = pl + P.K;  // keys any query of this stream can see
        const int tile_key0 = cc.tile * TK;

        ok = mbar_wait(&full_bar[st], ph, nullptr);
        if (!ok) break;
        // (debug build: the tile's rows lie inside the cache and the stage inside the warp's ring)
        if (!HAWK_IN_BOUNDS(P.dev_status, cc.row_base + tile_key0, static_cast<long long>(P.S) * P.H_kv * P.L_cap) ||
            !HAWK_IN_BOUNDS(P.dev_status, st, kStages))
            break;
        const uint32_t kbase = ring_u32 + st * kStageBytes;
        const uint32_t vbase = kbase + C::kHalves * C::kSubTileBytes;

        // ---- scores S^T = K Q^T for the whole tile
        float sc[NQT][KB][4];
#pragma unroll
        for (int kb = 0; kb < KB; ++kb) {
#pragma unroll
            for (int nq = 0; nq < NQT; ++nq) sc[nq][kb][0] = sc[nq][kb][1] = sc[nq][kb][2] = sc[nq][kb][3] = 0.f;
#pragma unroll
            for (int kk = 0; kk < DB; ++kk) {
                uint32_t ka[4];
                ldmatrix_x4(ka, kbase + kb * 2048 + k_off[kk]);
#pragma unroll
                for (int nq = 0; nq < NQT; ++nq) mma_bf16_16816(sc[nq][kb], ka, qb[nq][kk][0], qb[nq][kk][1]);
            }
        }
        // ---- causal mask inside the block, which also hides the cache rows past the last visible key
        if (tile_key0 + TK > pl) {
            // block rows visible to the queries in this thread's columns (bit m: row prefix + m); looked up here, at the
            // few tiles of an item that reach into the block, rather than carried in registers through all the others
            uint64_t qm[NQT][2];
#pragma unroll
            for (int nq = 0; nq < NQT; ++nq)
#pragma unroll
                for (int c = 0; c < 2; ++c) {
                    const int pos = (gr0 + nq * 8 + 2 * tq + c) % P.K;  // (padding rows get some position's mask)
                    qm[nq][c] = P.anc_mask ? P.anc_mask[pos] : chain_mask(pos);
                }
#pragma unroll
            for (int kb = 0; kb < KB; ++kb) {
                const int rel0 = tile_key0 + kb * 16 + g - pl, rel1 = rel0 + 8;
#pragma unroll
                for (int nq = 0; nq < NQT; ++nq) {
                    if (!key_visible(rel0, qm[nq][0])) sc[nq][kb][0] = -CUDART_INF_F;
                    if (!key_visible(rel0, qm[nq][1])) sc[nq][kb][1] = -CUDART_INF_F;
                    if (!key_visible(rel1, qm[nq][0])) sc[nq][kb][2] = -CUDART_INF_F;
                    if (!key_visible(rel1, qm[nq][1])) sc[nq][kb][3] = -CUDART_INF_F;
                }
            }
        }
        // ---- running softmax per query column (log2 domain): one max reduction and one rescale per tile
        uint32_t pb[NQT][KB][2];  // P^T as the 16 x 8 operand of the second product
#pragma unroll
        for (int nq = 0; nq < NQT; ++nq) {
            float mx0 = -CUDART_INF_F, mx1 = -CUDART_INF_F;
#pragma unroll
            for (int kb = 0; kb < KB; ++kb) {
                mx0 = fmaxf(mx0, fmaxf(sc[nq][kb][0], sc[nq][kb][2]));
                mx1 = fmaxf(mx1, fmaxf(sc[nq][kb][1], sc[nq][kb][3]));
            }
#pragma unroll
            for (int o = 4; o < 32; o <<= 1) {
                mx0 = fmaxf(mx0, __shfl_xor_sync(0xffffffffu, mx0, o));
                mx1 = fmaxf(mx1, __shfl_xor_sync(0xffffffffu, mx1, o));
            }
            const float mn0 = fmaxf(mrun[nq][0], mx0 * P.scale_log2), mn1 = fmaxf(mrun[nq][1], mx1 * P.scale_log2);
            const float mu0 = mn0 == -CUDART_INF_F ? 0.f : mn0, mu1 = mn1 == -CUDART_INF_F ? 0.f : mn1;
            const float a0 = fast_exp2(mrun[nq][0] - mu0), a1 = fast_exp2(mrun[nq][1] - mu1);
            mrun[nq][0] = mn0;
            mrun[nq][1] = mn1;
            float s0 = 0.f, s1 = 0.f;
#pragma unroll
            for (int kb = 0; kb < KB; ++kb) {
                const float p0 = fast_exp2(fmaf(sc[nq][kb][0], P.scale_log2, -mu0));
                const float p1 = fast_exp2(fmaf(sc[nq][kb][1], P.scale_log2, -mu1));
                const float p2 = fast_exp2(fmaf(sc[nq][kb][2], P.scale_log2, -mu0));
                const float p3 = fast_exp2(fmaf(sc[nq][kb][3], P.scale_log2, -mu1));
                s0 += p0 + p2;
                s1 += p1 + p3;
                // (key g / g+8) x (queries 2tq, 2tq+1)  ->  (keys 2tq, 2tq+1 / +8) x (query g)
                pb[nq][kb][0] = movmatrix_trans(pack_bf16(p0, p1));
                pb[nq][kb][1] = movmatrix_trans(pack_bf16(p2, p3));
            }
            lrun[nq][0] = lrun[nq][0] * a0 + s0;
            lrun[nq][1] = lrun[nq][1] * a1 + s1;
#pragma unroll
            for (int db = 0; db < DB; ++db) {
                ot[nq][db][0] *= a0;
                ot[nq][db][1] *= a1;
                ot[nq][db][2] *= a0;
                ot[nq][db][3] *= a1;
            }
        }
        // ---- O^T += V^T P^T.  Cache rows at or past n_total hold whatever the cache holds: zero
        // them so that 0 * NaN cannot appear.
        const bool ragged = tile_key0 + TK > n_total;
#pragma unroll
        for (int kb = 0; kb < KB; ++kb) {
            const int kleft = n_total - (tile_key0 + kb * 16);  // visible keys in this 16-key block
            if (ragged && kleft <= 0) break;
#pragma unroll
            for (int db = 0; db < DB; ++db) {
                uint32_t va[4];
                ldmatrix_x4_trans(va, vbase + kb * 2048 + v_off[db]);
                if (ragged && kleft < 16) {
                    // registers 0/1: keys 2tq, 2tq+1; registers 2/3: keys 2tq+8, 2tq+9 (low half = first key)
                    const int ka = 2 * tq, kb2 = 2 * tq + 8;
                    const uint32_t ma = (ka < kleft ? 0x0000ffffu : 0u) | (ka + 1 < kleft ? 0xffff0000u : 0u);
                    const uint32_t mb = (kb2 < kleft ? 0x0000ffffu : 0u) | (kb2 + 1 < kleft ? 0xffff0000u : 0u);
                    va[0] &= ma;
                    va[1] &= ma;
                    va[2] &= mb;
                    va[3] &= mb;
                }
#pragma unroll
                for (int nq = 0; nq < NQT; ++nq) mma_bf16_16816(ot[nq][db], va, pb[nq][kb][0], pb[nq][kb][1]);
            }
        }
        __syncwarp();
        --in_flight;
        // ---- the stage is free again: load the next tile of the share into it
        if (seek_valid<TK>(ci, f_end, P, flags)) {
            fence_proxy_async();  // the warp's reads of the stage come before the copy that overwrites it
            issue(ci, st);
            step<TK>(ci, f_end, P, flags);
            ++in_flight;
        }
        step<TK>(cc, f_end, P, flags);
        if (++st == kStages) {
            st = 0;
            ph ^= 1u;
        }
    }
    if (ok) {
        flush();
    } else {
        flags |= HAWK_DEV_TIMEOUT;
        // let the copies still in flight land (bounded) before the block can retire
        for (int i = 0; i < in_flight; ++i) {
            mbar_wait(&full_bar[st], ph, nullptr);
            if (++st == kStages) {
                st = 0;
                ph ^= 1u;
            }
        }
    }
    if (flags && lane == 0 && P.dev_status) atomicOr(P.dev_status, flags);

    if (grouped) {
        // ---- the G warps of an item sit side by side in this block: fold their partial results, in share
        // order, straight from shared memory (no workspace, no merge kernel)
        __syncthreads();
        constexpr int PER = D / 32;
        const int G = P.group_g, ipb = kWarps / G;
        const int total = ipb * P.rows_per_item;
        for (int idx = warp; idx < total; idx += kWarps) {
            const int il = idx / P.rows_per_item, r = idx - il * P.rows_per_item;
            const int item = static_cast<int>(blockIdx.x) * ipb + il;
            if (item >= P.items) break;
            int it = item;
            const int chunk = it % P.chunks;
            it /= P.chunks;
            const int hk = it % P.H_kv, s = it / P.H_kv;
            if (r >= min(P.rows_per_item, group * P.K - chunk * P.rows_per_item)) continue;
            float acc[PER];
#pragma unroll
            for (int c = 0; c < PER; ++c) acc[c] = 0.f;
            float mm = -CUDART_INF_F, ll = 0.f;
            for (int gg = 0; gg < G; ++gg) {
                const int wg = il * G + gg;
                if (!has_part[wg]) continue;  // that share lay past the stream's last visible key
                const float *ps = reinterpret_cast<const float *>(smem + wg * kStages * kStageBytes);
                const float2 m_l = *reinterpret_cast<const float2 *>(ps + P.rows_per_item * D + 2 * r);
                const float mn = fmaxf(mm, m_l.x);
                const float mu = mn == -CUDART_INF_F ? 0.f : mn;
                const float f_old = fast_exp2(mm - mu), f_new = fast_exp2(m_l.x - mu);
                mm = mn;
                ll = ll * f_old + m_l.y * f_new;
#pragma unroll
                for (int c = 0; c < PER; ++c) acc[c] = acc[c] * f_old + ps[r * D + lane * PER + c] * f_new;
            }
            const float inv = 1.f / ll;
            const int gr = chunk * P.rows_per_item + r;
            const int h = hk * group + gr / P.K, i = gr % P.K;
            __nv_bfloat16 *dst = P.out + ((static_cast<size_t>(s) * P.K + i) * P.H + h) * D + lane * PER;
#pragma unroll
            for (int c = 0; c < PER; c += 2)
                *reinterpret_cast<__nv_bfloat162 *>(dst + c) = __floats2bfloat162_rn(acc[c] * inv, acc[c + 1] * inv);
        }
    }
}

// Division of a 31-bit unsigned number by a divisor fixed at launch: one multiply-high and a shift
// (division by invariant integers, Granlund and Montgomery): mul = ceil(2^(31 + ceil(log2 d)) / d),
// n / d = umulhi(n, mul) >> (ceil(log2 d) - 1) for 0 <= n < 2^31.  The host fills it in.
struct FastDiv {
    uint32_t d, mul, shr;
    __host__ void set(uint32_t div)
    {
        d = div;
        if (div <= 1) {
            mul = 0;
            shr = 0;
            return;
        }
        uint32_t lg = 0;
        while ((1u << lg) < div) ++lg;  // ceil(log2 div), 1..31
        const unsigned long long pw = 1ull << (31 + lg);
        mul = static_cast<uint32_t>((pw + div - 1) / div);
        shr = lg - 1;
    }
    __device__ __forceinline__ uint32_t div(uint32_t n) const { return d <= 1 ? n : __umulhi(n, mul) >> shr; }
    __device__ __forceinline__ uint32_t divmod(uint32_t n, uint32_t &rem) const
    {
        const uint32_t q = div(n);
        rem = n - q * d;
        return q;
    }
};

// Divisors of the merge kernel's index arithmetic.
struct MergeDivs {
    FastDiv workers, total, tiles_per_item, chunks, h_kv, rows_per_item, k;
};

// Index arithmetic of the merge kernel: which item a unit stands for, the shares its tiles went to and
// where their partial results are.  Two forms: 32-bit with launch-time divisors when every product of
// a tile index and the worker count fits 31 bits (a dozen divisions by run-time values would otherwise
// be most of the kernel's instructions), plain 64-bit otherwise.
template <int AHEAD>
struct MergeIndex {
    bool cut;  // this unit stands for an item whose tiles were spread over several shares
    int item, g_first, g_last, s, hk, chunk;
    int seg_off[AHEAD];  // first tile, inside the item, of contribution t
    int slot_id[AHEAD];  // its partial slot: share * 2 + (0 head of the share, 1 tail)
};

template <int AHEAD>
__device__ __forceinline__ void merge_index32(const AttnParams &P, const MergeDivs &dv, int unit, int units,
                                              int by_boundary, MergeIndex<AHEAD> &ix)
{
    const uint32_t T = static_cast<uint32_t>(P.total_tiles), W = static_cast<uint32_t>(P.workers);
    const uint32_t tpi = static_cast<uint32_t>(P.tiles_per_item);
    auto begin_of = [&](uint32_t g) { return dv.workers.div(g * T); };
    auto owner_of = [&](uint32_t f) { return dv.total.div((f + 1) * W - 1); };
    uint32_t item = static_cast<uint32_t>(unit);
    bool first_inside = true;
    if (by_boundary && unit < units) {
        const uint32_t sb = begin_of(static_cast<uint32_t>(unit) + 1);
        item = dv.tiles_per_item.div(sb);
        const uint32_t ia = item * tpi;
        first_inside = sb > ia && (unit == 0 || begin_of(static_cast<uint32_t>(unit)) <= ia);
    }
    ix.cut = unit < units && first_inside;
    ix.item = static_cast<int>(item);
    ix.g_first = ix.g_last = ix.s = ix.hk = ix.chunk = 0;
    const uint32_t a = item * tpi, b = a + tpi;
    if (ix.cut) {
        ix.g_first = static_cast<int>(owner_of(a));
        ix.g_last = static_cast<int>(owner_of(b - 1));
        uint32_t chunk, hk;
        const uint32_t it = dv.chunks.divmod(item, chunk);
        ix.s = static_cast<int>(dv.h_kv.divmod(it, hk));
        ix.hk = static_cast<int>(hk);
        ix.chunk = static_cast<int>(chunk);
        ix.cut = ix.g_first != ix.g_last;
    }
#pragma unroll
    for (int t = 0; t < AHEAD; ++t) {
        const int gg = min(ix.g_first + t, ix.g_last);
        const uint32_t sb = begin_of(static_cast<uint32_t>(gg));
        ix.seg_off[t] = static_cast<int>((sb > a ? sb : a) - a);
        ix.slot_id[t] = gg * 2 + (a <= sb ? 0 : 1);
    }
}

template <int AHEAD>
__device__ __forceinline__ void merge_index64(const AttnParams &P, int unit, int units, int by_boundary,
                                              MergeIndex<AHEAD> &ix)
{
    const long long T = P.total_tiles, tpi = P.tiles_per_item;
    long long item = unit;
    bool first_inside = true;
    if (by_boundary && unit < units) {
        const long long sb = share_begin(unit + 1, T, P.workers);
        item = sb / tpi;
        const long long ia = item * tpi;
        first_inside = sb > ia && (unit == 0 || share_begin(unit, T, P.workers) <= ia);
    }
    ix.cut = unit < units && first_inside;
    ix.item = static_cast<int>(item);
    ix.g_first = ix.g_last = ix.s = ix.hk = ix.chunk = 0;
    const long long a = item * tpi, b = a + tpi;
    if (ix.cut) {
        ix.g_first = owner(a, T, P.workers);
        ix.g_last = owner(b - 1, T, P.workers);
        int it = ix.item;
        ix.chunk = it % P.chunks;
        it /= P.chunks;
        ix.hk = it % P.H_kv;
        ix.s = it / P.H_kv;
        ix.cut = ix.g_first != ix.g_last;
    }
#pragma unroll
    for (int t = 0; t < AHEAD; ++t) {
        const int gg = min(ix.g_first + t, ix.g_last);
        const long long sb = share_begin(gg, T, P.workers);
        ix.seg_off[t] = static_cast<int>((sb > a ? sb : a) - a);
        ix.slot_id[t] = gg * 2 + (a <= sb ? 0 : 1);
    }
}

// Merges the partial results of every item whose tiles were spread over several shares:
// one warp per (item, query row of the item), lanes across the head dimension.  All index
// arithmetic and the loads of the call's inputs come before the wait on the attention kernel; after
// it the loads of up to kAhead contributions are issued together, so the kernel adds one memory
// round trip to the call.
// The grid runs over `units`: the items themselves, or (by_boundary) the share boundaries 1 .. workers-1
// when there are fewer of those than items; a boundary stands for the item it falls into, if it is the
// first one strictly inside that item, so every cut item is merged exactly once and the grid stays
// within one wave however many items the call has.
// kAhead = 2 (an item never spans more than two shares: the common case when items are shorter than
// shares) keeps the kernel within 32 registers, so that eight blocks fit an SM and the grid is one wave.
template <int D, int kAhead>
__global__ void __launch_bounds__(256, kAhead <= 2 ? 8 : 4)
    attn_combine_kernel(const AttnParams P, const MergeDivs dv, int units, int by_boundary)
{
    constexpr int TK = AttnCfg<D>::kTileKeys;
    constexpr int PER = D / 32;
    allow_dependent_launch();
    const int wid = (blockIdx.x * blockDim.x + threadIdx.x) >> 5;
    const int lane = threadIdx.x & 31;
    uint32_t r_u;
    const int unit = static_cast<int>(dv.rows_per_item.divmod(static_cast<uint32_t>(wid), r_u));
    const int r = static_cast<int>(r_u);
    const long long T = P.total_tiles;
    MergeIndex<kAhead> ix;
    if (P.idx32)  // block-uniform
        merge_index32<kAhead>(P, dv, unit, units, by_boundary, ix);
    else
        merge_index64<kAhead>(P, unit, units, by_boundary, ix);
    const long long a = static_cast<long long>(ix.item) * P.tiles_per_item;
    const int g_first = ix.g_first, g_last = ix.g_last, s = ix.s, hk = ix.hk, chunk = ix.chunk;
    const int group = P.H / P.H_kv;
    // one share held the whole item and wrote the result itself; rows past the item's last do not exist
    const bool active = ix.cut && r < min(P.rows_per_item, group * P.K - chunk * P.rows_per_item);
    // tile offset inside the item at which each contribution starts, and where it is stored
    const float *slot[kAhead];
    int seg_off[kAhead];
#pragma unroll
    for (int t = 0; t < kAhead; ++t) {
        seg_off[t] = ix.seg_off[t];
        slot[t] = P.part + static_cast<size_t>(ix.slot_id[t]) * P.rows_per_item * (D + 2);
    }
    const int pl_raw = active ? P.prefix_len[s] : 0;  // an input of the call: readable before the wait
    grid_dependency_wait();  // every thread waits, so this grid cannot retire before the attention kernel has
    if (!active) return;

    float2 ml[kAhead];
    float v[kAhead][PER];
#pragma unroll
    for (int t = 0; t < kAhead; ++t) {  // slots always exist; which of them were written is decided below
        ml[t] = *reinterpret_cast<const float2 *>(slot[t] + P.rows_per_item * D + 2 * r);
        const float *ps = slot[t] + r * D + lane * PER;
        if constexpr (PER == 2) {
            const float2 x = *reinterpret_cast<const float2 *>(ps);
            v[t][0] = x.x;
            v[t][1] = x.y;
        } else {
            const float4 x = *reinterpret_cast<const float4 *>(ps);
            v[t][0] = x.x;
            v[t][1] = x.y;
            v[t][PER - 2] = x.z;
            v[t][PER - 1] = x.w;
        }
    }
    const int ntiles = (max(0, min(pl_raw, P.pl_max)) + P.K + TK - 1) / TK;

    float acc[PER];
#pragma unroll
    for (int c = 0; c < PER; ++c) acc[c] = 0.f;
    float mm = -CUDART_INF_F, ll = 0.f;
    auto fold = [&](float2 m_l, const float (&val)[PER]) {
        const float mn = fmaxf(mm, m_l.x);
        const float mu = mn == -CUDART_INF_F ? 0.f : mn;
        const float f_old = fast_exp2(mm - mu), f_new = fast_exp2(m_l.x - mu);
        mm = mn;
        ll = ll * f_old + m_l.y * f_new;
#pragma unroll
        for (int c = 0; c < PER; ++c) acc[c] = acc[c] * f_old + val[c] * f_new;
    };
    // a share whose part of the item starts past the stream's last visible key wrote nothing
#pragma unroll
    for (int t = 0; t < kAhead; ++t)
        if (g_first + t <= g_last && seg_off[t] < ntiles) fold(ml[t], v[t]);
    for (int gg = g_first + kAhead; gg <= g_last; ++gg) {  // items spread over more shares than that: one by one
        const long long sb = share_begin(gg, T, P.workers);
        if ((sb > a ? sb : a) - a >= ntiles) break;
        const float *sl = P.part + (static_cast<size_t>(gg) * 2 + (a <= sb ? 0 : 1)) * P.rows_per_item * (D + 2);
        const float2 m_l = *reinterpret_cast<const float2 *>(sl + P.rows_per_item * D + 2 * r);
        float val[PER];
#pragma unroll
        for (int c = 0; c < PER; ++c) val[c] = sl[r * D + lane * PER + c];
        fold(m_l, val);
    }
    const float inv = 1.f / ll;
    const int gr = chunk * P.rows_per_item + r;
    uint32_t i_u;
    const int h = hk * group + static_cast<int>(dv.k.divmod(static_cast<uint32_t>(gr), i_u)), i = static_cast<int>(i_u);
    __nv_bfloat16 *dst = P.out + ((static_cast<size_t>(s) * P.K + i) * P.H + h) * D + lane * PER;
#pragma unroll
    for (int c = 0; c < PER; c += 2)
        *reinterpret_cast<__nv_bfloat162 *>(dst + c) = __floats2bfloat162_rn(acc[c] * inv, acc[c + 1] * inv);
}

struct AttnPlan {
    int chunks, items, rows_per_item, tiles_per_item, workers, grid;
    bool whole;  // one warp per item (3 warps x 8 stages per block) instead of equal shares (8 x 3)
    int group_g;  // > 0: every item split evenly over this many warps of a 4-warp block and merged there
    long long total_tiles;
    bool any_cut;  // some item's tiles are spread over more than one share: partials + merge kernel needed
};

// Launch shape from host-known sizes only, so that the workspace query and the launch agree.
AttnPlan make_plan(int S, int K, int H, int H_kv, int D, int max_prefix_len)
{
    AttnPlan pl;
    const int group = H / H_kv;
    const int total_rows = group * K;            // (head of the group, position) pairs sharing one kv head
    const int rows_max = D == 64 ? 32 : 24;      // what one warp's registers hold
    pl.chunks = (total_rows + rows_max - 1) / rows_max;
    pl.rows_per_item = ((total_rows + pl.chunks - 1) / pl.chunks + 7) / 8 * 8;
    pl.items = S * H_kv * pl.chunks;
    const int tk = D == 64 ? AttnCfg<64>::kTileKeys : AttnCfg<128>::kTileKeys;
    pl.tiles_per_item = (max_prefix_len + K + tk - 1) / tk;
    pl.total_tiles = static_cast<long long>(pl.items) * pl.tiles_per_item;
    pl.whole = pl.items <= kPlanSms * kWarpsWhole && pl.tiles_per_item <= kWholeMaxTiles;
    // few long items of one 8-row column tile (a kernel of under 170 registers, three 4-warp blocks per SM): split
    // each evenly over the 4 warps of a block if all blocks are resident at once; the warps fold their partial
    // results in shared memory and nothing is left for a merge kernel
    pl.group_g = 0;
    // (with fewer than 222 items the 4 warps per item are fewer than three quarters of the shares' 1184 workers:
    // long items then go faster as shares)
#ifndef HAWK_ATTN_GROUP_MAX_ROWS
#define HAWK_ATTN_GROUP_MAX_ROWS 8
#endif
    if (pl.rows_per_item <= HAWK_ATTN_GROUP_MAX_ROWS && 4 * pl.items >= 3 * kPlanSms * 2 && pl.items <= 3 * kPlanSms &&
        pl.tiles_per_item >= 2 * kWarpsGroup) {
        pl.group_g = kWarpsGroup;
        pl.whole = false;  // (from 8 tiles on, four warps with a merge in shared memory beat one warp alone)
    }
    if (pl.whole) {
        pl.workers = pl.items;  // share g = item g
        pl.grid = pl.items < kPlanSms ? pl.items : kPlanSms;
    } else if (pl.group_g > 0) {
        pl.workers = pl.items * pl.group_g;  // share w = part (w % G) of item (w / G)
        pl.grid = (pl.workers + kWarpsGroup - 1) / kWarpsGroup;
    } else {
        const long long cap = static_cast<long long>(kPlanSms) * kWarpsShares;
        pl.workers = static_cast<int>(pl.total_tiles < cap ? pl.total_tiles : cap);
        pl.grid = (pl.workers + kWarpsShares - 1) / kWarpsShares;
    }
    pl.any_cut = false;
    for (int it = 0; it < pl.items && !pl.any_cut && pl.group_g == 0; ++it) {
        const long long a = static_cast<long long>(it) * pl.tiles_per_item, b = a + pl.tiles_per_item;
        pl.any_cut = owner(a, pl.total_tiles, pl.workers) != owner(b - 1, pl.total_tiles, pl.workers);
    }
    return pl;
}

template <int D, int NQT, int WARPS, int STAGES>
cudaError_t launch_attn_shape(const CUtensorMap &map_k, const CUtensorMap &map_v, const AttnParams &P, int grid,
                              cudaStream_t st)
{
    constexpr size_t smem = AttnCfg<D>::smem_bytes(WARPS, STAGES);
    int device = 0;
    cudaError_t e = cudaGetDevice(&device);
    if (e != cudaSuccess) return e;
    if (device < 0 || device >= 64) return cudaErrorInvalidDevice;
    static std::atomic<unsigned long long> attr_done{0};  // one bit per device: the limit is a per-device attribute of the function
    if (!((attr_done.load(std::memory_order_relaxed) >> device) & 1ull)) {
        e = cudaFuncSetAttribute(attn_kernel<D, NQT, WARPS, STAGES>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                 static_cast<int>(smem));
        if (e != cudaSuccess) return e;
        attr_done.fetch_or(1ull << device, std::memory_order_relaxed);
    }
    return hawk_host::launch_dependent(attn_kernel<D, NQT, WARPS, STAGES>, dim3(grid), dim3(WARPS * 32), smem, st, map_k,
                                       map_v, P);
}

template <int D, int NQT>
cudaError_t launch_attn(const CUtensorMap &map_k, const CUtensorMap &map_v, const AttnParams &P, int grid, bool whole,
                        cudaStream_t st)
{
    if (P.group_g > 0) return launch_attn_shape<D, NQT, kWarpsGroup, kStagesGroup>(map_k, map_v, P, grid, st);
    return whole ? launch_attn_shape<D, NQT, kWarpsWhole, kStagesWhole>(map_k, map_v, P, grid, st)
                 : launch_attn_shape<D, NQT, kWarpsShares, kStagesShares>(map_k, map_v, P, grid, st);
}

}  // namespace

extern "C" size_t hawk_verify_attn_workspace_bytes(int S, int K, int H, int H_kv, int D, int max_prefix_len)
{
    if (S <= 0 || K < 1 || K > 64 || H <= 0 || H_kv <= 0 || H % H_kv != 0 || (D != 64 && D != 128) ||
        max_prefix_len < 0)
        return 0;
    const AttnPlan pl = make_plan(S, K, H, H_kv, D, max_prefix_len);
    if (!pl.any_cut) return 0;
    return static_cast<size_t>(pl.workers) * 2 * pl.rows_per_item * (D + 2) * sizeof(float);
}

hawk_status hawk_host::check_verify_attn_args(const void *q, const void *k_cache, const void *v_cache,
                                              const int32_t *prefix_len, const void *out, int S, int K, int H, int H_kv,
                                              int D, int L_cap, int max_prefix_len, float sm_scale,
                                              const void *workspace, size_t workspace_bytes)
{
    if (S < 0 || K < 0 || H < 0 || H_kv < 0 || D < 0 || L_cap < 0 || max_prefix_len < 0) return HAWK_ERR_SHAPE;
    if (S == 0) return HAWK_OK;
    if (!q || !k_cache || !v_cache || !prefix_len || !out) return HAWK_ERR_NULL;
    if (K < 1 || K > 64 || (D != 64 && D != 128) || H < 1 || H_kv < 1 || H % H_kv != 0) return HAWK_ERR_UNSUPPORTED;
    if (max_prefix_len + K > L_cap) return HAWK_ERR_SHAPE;
    if (static_cast<long long>(S) * H_kv * L_cap >= (1ll << 31)) return HAWK_ERR_UNSUPPORTED;
    if (!(sm_scale > 0.f) || isinf(sm_scale)) return HAWK_ERR_PARAM;
    if (!hawk_host::aligned16(q) || !hawk_host::aligned16(k_cache) || !hawk_host::aligned16(v_cache) ||
        !hawk_host::aligned16(out))
        return HAWK_ERR_ALIGN;
    const size_t need = hawk_verify_attn_workspace_bytes(S, K, H, H_kv, D, max_prefix_len);
    if (need > 0) {
        if (!workspace || workspace_bytes < need) return HAWK_ERR_WORKSPACE;
        if (!hawk_host::aligned16(workspace)) return HAWK_ERR_ALIGN;
    }
    return HAWK_OK;
}

namespace {

// Common body of hawk_verify_attn (anc_mask == NULL: causal block) and hawk_verify_attn_tree.
hawk_status verify_attn_impl(const void *q, const void *k_cache, const void *v_cache, const int32_t *prefix_len,
                             const uint64_t *anc_mask, void *out, int S, int K, int H, int H_kv, int D, int L_cap,
                             int max_prefix_len, float sm_scale, void *workspace, size_t workspace_bytes,
                             int32_t *dev_status, hawk_stream_t stream)
{
    const hawk_status chk = hawk_host::check_verify_attn_args(q, k_cache, v_cache, prefix_len, out, S, K, H, H_kv, D, L_cap,
                                                             max_prefix_len, sm_scale, workspace, workspace_bytes);
    if (chk != HAWK_OK) return chk;
    if (S == 0) return HAWK_OK;
    if (!hawk_host::is_sm100(nullptr)) return HAWK_ERR_UNSUPPORTED;
    const AttnPlan pl = make_plan(S, K, H, H_kv, D, max_prefix_len);

    const int tile_keys = D == 64 ? AttnCfg<64>::kTileKeys : AttnCfg<128>::kTileKeys;
    CUtensorMap map_k, map_v;
    const uint64_t rows = static_cast<uint64_t>(S) * H_kv * L_cap;
    if (!hawk_host::encode_bf16_rows_sw128(&map_k, k_cache, rows, D, tile_keys, true) ||
        !hawk_host::encode_bf16_rows_sw128(&map_v, v_cache, rows, D, tile_keys, true))
        return HAWK_ERR_CUDA;

    AttnParams P;
    P.q = static_cast<const __nv_bfloat16 *>(q);
    P.prefix_len = prefix_len;
    P.out = static_cast<__nv_bfloat16 *>(out);
    P.part = static_cast<float *>(workspace);
    P.S = S;
    P.K = K;
    P.H = H;
    P.H_kv = H_kv;
    P.L_cap = L_cap;
    P.pl_max = max_prefix_len < L_cap - K ? max_prefix_len : L_cap - K;
    P.anc_mask = anc_mask;
    P.rows_per_item = pl.rows_per_item;
    P.chunks = pl.chunks;
    P.tiles_per_item = pl.tiles_per_item;
    P.workers = pl.workers;
    P.total_tiles = pl.total_tiles;
    P.group_g = pl.group_g;
    P.items = pl.items;
    P.idx32 = (pl.total_tiles + 1) * pl.workers < (1ll << 31) ? 1 : 0;
    P.scale_log2 = sm_scale * 1.4426950408889634f;
    P.dev_status = dev_status;

    cudaStream_t st = reinterpret_cast<cudaStream_t>(stream);
    const int nqt = pl.rows_per_item / 8;  // 8-query column tiles per item: 1..4 (D = 64), 1..3 (D = 128)
    cudaError_t err = cudaErrorInvalidValue;
    if (D == 64) {
        if (nqt == 1) err = launch_attn<64, 1>(map_k, map_v, P, pl.grid, pl.whole, st);
        else if (nqt == 2) err = launch_attn<64, 2>(map_k, map_v, P, pl.grid, pl.whole, st);
        else if (nqt == 3) err = launch_attn<64, 3>(map_k, map_v, P, pl.grid, pl.whole, st);
        else if (nqt == 4) err = launch_attn<64, 4>(map_k, map_v, P, pl.grid, pl.whole, st);
    } else {
        if (nqt == 1) err = launch_attn<128, 1>(map_k, map_v, P, pl.grid, pl.whole, st);
        else if (nqt == 2) err = launch_attn<128, 2>(map_k, map_v, P, pl.grid, pl.whole, st);
        else if (nqt == 3) err = launch_attn<128, 3>(map_k, map_v, P, pl.grid, pl.whole, st);
    }
    if (err != cudaSuccess) return HAWK_ERR_CUDA;
    if (pl.any_cut) {
        const int threads = 256;
        const int by_boundary = pl.items > pl.workers - 1 ? 1 : 0;
        const int units = by_boundary ? pl.workers - 1 : pl.items;
        const long long warps = static_cast<long long>(units) * pl.rows_per_item;
        const int blocks = static_cast<int>((warps * 32 + threads - 1) / threads);
        MergeDivs dv;
        dv.workers.set(static_cast<uint32_t>(pl.workers));
        dv.total.set(P.idx32 ? static_cast<uint32_t>(pl.total_tiles) : 1u);
        dv.tiles_per_item.set(static_cast<uint32_t>(pl.tiles_per_item));
        dv.chunks.set(static_cast<uint32_t>(pl.chunks));
        dv.h_kv.set(static_cast<uint32_t>(P.H_kv));
        dv.rows_per_item.set(static_cast<uint32_t>(pl.rows_per_item));
        dv.k.set(static_cast<uint32_t>(P.K));
        // shares hold floor(T / workers) tiles or one more: an item no longer than the shorter kind meets at
        // most one share boundary
        // shares hold floor(T / workers) tiles or one more: an item of t tiles meets at most ceil(t / floor) share
        // boundaries, i.e. has at most that many contributions plus one; all of them are loaded at once
        const long long min_share = pl.total_tiles / pl.workers;
        const long long contrib = min_share > 0 ? (pl.tiles_per_item + min_share - 1) / min_share + 1 : 9;
        auto kernel = D == 64 ? (contrib <= 2 ? attn_combine_kernel<64, 2>
                                 : contrib <= 4 ? attn_combine_kernel<64, 4> : attn_combine_kernel<64, 8>)
                              : (contrib <= 2 ? attn_combine_kernel<128, 2>
                                 : contrib <= 4 ? attn_combine_kernel<128, 4> : attn_combine_kernel<128, 8>);
        err = hawk_host::launch_dependent(kernel, dim3(blocks), dim3(threads), 0, st, P, dv, units, by_boundary);
        if (err != cudaSuccess) return HAWK_ERR_CUDA;
    }
    return HAWK_OK;
}

}  // namespace

extern "C" hawk_status hawk_verify_attn(const void *q, const void *k_cache, const void *v_cache,
                                        const int32_t *prefix_len, void *out, int S, int K, int H, int H_kv, int D,
                                        int L_cap, int max_prefix_len, float sm_scale, void *workspace,
                                        size_t workspace_bytes, int32_t *dev_status, hawk_stream_t stream)
{
    const hawk_host::NvtxRange nvtx_range("hawk_verify_attn");
    return verify_attn_impl(q, k_cache, v_cache, prefix_len, nullptr, out, S, K, H, H_kv, D, L_cap, max_prefix_len,
                            sm_scale, workspace, workspace_bytes, dev_status, stream);
}

extern "C" hawk_status hawk_verify_attn_tree(const void *q, const void *k_cache, const void *v_cache,
                                             const int32_t *prefix_len, const uint64_t *anc_mask, void *out, int S,
                                             int N, int H, int H_kv, int D, int L_cap, int max_prefix_len,
                                             float sm_scale, void *workspace, size_t workspace_bytes,
                                             int32_t *dev_status, hawk_stream_t stream)
{
    const hawk_host::NvtxRange nvtx_range("hawk_verify_attn_tree");
    if (S > 0 && !anc_mask) return HAWK_ERR_NULL;
    return verify_attn_impl(q, k_cache, v_cache, prefix_len, anc_mask, out, S, N, H, H_kv, D, L_cap, max_prefix_len,
                            sm_scale, workspace, workspace_bytes, dev_status, stream);
}
