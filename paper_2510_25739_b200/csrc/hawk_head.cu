// hawk_head_proj: logits[m][v] = sum_c x[m][c] * w[v][c] on the 5th-generation tensor cores.
//
// The token codebook sits on the MMA's M dimension (128 weight rows per tile) and the token rows on
// N (16..256), so a handful of draft positions wastes nothing: the instruction's N simply shrinks.
// Both operands are K-major exactly as stored, so TMA drops [rows][64 columns] boxes with the
// 128-byte swizzle into shared memory and tcgen05.mma reads them through matrix descriptors.
//
// One persistent block per SM, warp-specialised:
//   warp 0      TMA producer: W box (128 x 64) + X box (BN x 64) per stage, full/empty mbarriers
//   warp 1      allocates TMEM, issues tcgen05.mma (one lane), commits stages and accumulators
//   warps 2..5  epilogue: tcgen05.ld of the fp32 accumulator (lane = token id, column = token row),
//               coalesced 128-byte stores into logits[token][vocab]
// The accumulator is double-buffered in TMEM so the epilogue of one tile overlaps the MMAs of the next.
//
// hawk_head_proj_cfg runs the same kernel with the two guidance streams of a position side by side in
// one tile: columns [0, BN/2) hold conditional token rows, columns [BN/2, BN) the unconditional rows of
// the same (sequence, position) pairs (two X boxes per stage).  The epilogue combines the two
// accumulators of a pair (subtract, fused multiply-add, divide: the arithmetic of the accept kernels)
// and writes ONE row of guided logits, so the logits cross HBM half as often on the way out and half
// as often on the way into the accept stage.
#include <atomic>

#include "hawk_common.cuh"

namespace {

using namespace hawk;

constexpr int kBM = 128;  // weight rows (token ids) per tile = MMA M
constexpr int kBK = 64;   // bf16 columns per stage = 128 bytes = one swizzle span
constexpr int kHeadThreads = 192;
constexpr int kATileBytes = kBM * kBK * 2;  // 16 KB
constexpr int kMaxStages = 12;
constexpr uint32_t kTmemCols = 512;

struct HeadParams {
    float *logits;
    int M, hidden, V, v_begin, v_end;
    int BN;        // token rows per tile (multiple of 16, <= 256)
    int tiles_m;   // vocab tiles
    int tiles_n;   // token tiles
    int stages;
    int stage_bytes;
    int wide;      // pair kernel: one accumulator of BN (up to 512) columns, every k-step as two MMAs of BN / 2 columns
    int ksplit;    // 1, or 2: a pair of blocks per tile, each over half of the hidden dimension; block 1 hands its sums to block 0
    int xchg_off;  // ksplit == 2: byte offset, in a block's shared memory, of the buffer that receives the partner's sums
    int pairs;     // 0: plain logits; > 0: guided logits of this many (sequence, position) pairs
    float cfg_scale, temperature;
    int32_t *dev_status;
};

// Epilogue of one tile for one thread: the thread owns token id v (its tensor-memory lane) and walks
// the tile's token columns 16 at a time; lanes of a warp hold consecutive ids, so every store
// instruction writes 128 contiguous bytes of one logits row.
// Warps that share a lane quarter split the 16-column chunks among themselves (chunk0, chunk_step).
// WIDE (pair kernel, two MMAs of BN / 2 columns per k-step): accumulator column t of MMA half c = t / (BN / 2)
// comes from CTA (t % (BN / 2)) / (BN / 4), row c * (BN / 4) + t % (BN / 4) of that CTA's token rows; BN is a
// multiple of 64 there, so a 16-column chunk never straddles two of these ranges.
// r += the partner block's sums for 16-column chunk `col / 16` of accumulator row `row` (own + partner, in that order).
__device__ __forceinline__ void add_partner(uint32_t (&r)[16], const float *partner, int col, int row)
{
    const float4 *src = reinterpret_cast<const float4 *>(partner + (static_cast<size_t>(col >> 4) * kBM + row) * 16);
#pragma unroll
    for (int q = 0; q < 4; ++q) {
        const float4 a = src[q];
        r[4 * q + 0] = __float_as_uint(__fadd_rn(__uint_as_float(r[4 * q + 0]), a.x));
        r[4 * q + 1] = __float_as_uint(__fadd_rn(__uint_as_float(r[4 * q + 1]), a.y));
        r[4 * q + 2] = __float_as_uint(__fadd_rn(__uint_as_float(r[4 * q + 2]), a.z));
        r[4 * q + 3] = __float_as_uint(__fadd_rn(__uint_as_float(r[4 * q + 3]), a.w));
    }
}

// KSPLIT: `partner` holds the other block's sums over its half of the hidden dimension, 16-column chunk k of
// accumulator row `row` at partner[(k * 128 + row) * 16 ..]; they are added to this block's (this + partner, always
// in that order) before anything else happens to the value.
template <bool KSPLIT = false, bool WIDE = false>
__device__ __forceinline__ void epilogue_store(const HeadParams &P, uint32_t taddr, int tn, int v, bool v_ok,
                                               int chunk0 = 0, int chunk_step = 1, const float *partner = nullptr,
                                               int row = 0)
{
    if (P.pairs == 0) {
        const int n0 = tn * P.BN;
        for (int c = 16 * chunk0; c < P.BN; c += 16 * chunk_step) {
            uint32_t r[16];
            tmem_ld_32x16(taddr + c, r);
            tmem_ld_wait();
            if constexpr (KSPLIT) add_partner(r, partner, c, row);
            int nbase = n0 + c;
            if constexpr (WIDE) {
                const int half = P.BN / 2, quarter = P.BN / 4;
                const int mma = c / half, j = c - mma * half;
                nbase = n0 + (j / quarter) * half + mma * quarter + j % quarter;
            }
            if (v_ok) {
#pragma unroll
                for (int j = 0; j < 16; ++j) {
                    const int n = nbase + j;
                    if (n < P.M && HAWK_IN_BOUNDS(P.dev_status, v, P.V)) {
                        float *dst = &P.logits[static_cast<size_t>(n) * P.V + v];
                        *dst = __uint_as_float(r[j]);
                    }
                }
            }
        }
    } else {
        const int half = P.BN / 2;  // pairs per tile, a multiple of 16
        const bool unit_T = P.temperature == 1.0f;
        for (int c = 16 * chunk0; c < half; c += 16 * chunk_step) {
            uint32_t rc[16], ru[16];
            // columns of pairs c .. c + 15: conditional rows, then unconditional rows; WIDE: MMA half m = c / (BN / 4)
            // holds the conditional rows of its pairs in its first BN / 4 columns, the unconditional ones in the rest
            int col_c = c, col_u = half + c;
            if constexpr (WIDE) {
                const int quarter = P.BN / 4, m = c / quarter, jj = c - m * quarter;
                col_c = m * half + jj;
                col_u = col_c + quarter;
            }
            tmem_ld_32x16(taddr + col_c, rc);
            tmem_ld_32x16(taddr + col_u, ru);
            tmem_ld_wait();
            if constexpr (KSPLIT) {
                add_partner(rc, partner, col_c, row);
                add_partner(ru, partner, col_u, row);
            }
            if (v_ok) {
#pragma unroll
                for (int j = 0; j < 16; ++j) {
                    const int pair = tn * half + c + j;
                    const float lc = __uint_as_float(rc[j]), lu = __uint_as_float(ru[j]);
                    float g = __fmaf_rn(P.cfg_scale, __fsub_rn(lc, lu), lu);
                    if (!unit_T) g = __fdiv_rn(g, P.temperature);
                    if (pair < P.pairs && HAWK_IN_BOUNDS(P.dev_status, v, P.V)) P.logits[static_cast<size_t>(pair) * P.V + v] = g;
                }
            }
        }
    }
}

// A block of a pair hands the accumulator chunks that its partner will finish (this thread's row of them) to the
// partner's exchange buffer.  Ownership alternates by 16-column chunk: plain logits, chunk k belongs to block k % 2;
// guided logits, the chunks of pairs 16k .. 16k + 15 (their conditional and their unconditional columns) to block k % 2.
__device__ __forceinline__ void epilogue_send(const HeadParams &P, uint32_t taddr, int row, uint32_t partner_buf, int partner)
{
    const int half = P.BN / 2;
    for (int c = 0; c < P.BN; c += 16) {
        const int owner = ((P.pairs == 0 ? c : c % half) >> 4) & 1;
        if (owner != partner) continue;
        uint32_t r[16];
        tmem_ld_32x16(taddr + c, r);
        tmem_ld_wait();
        const uint32_t dst = partner_buf + static_cast<uint32_t>(((c >> 4) * kBM + row) * 64);
#pragma unroll
        for (int q = 0; q < 4; ++q)
            asm volatile("st.shared::cluster.v4.b32 [%0], {%1, %2, %3, %4};" ::"r"(dst + 16 * q), "r"(r[4 * q]), "r"(r[4 * q + 1]),
                         "r"(r[4 * q + 2]), "r"(r[4 * q + 3])
                         : "memory");
    }
}

// One block per tile of 128 token ids x BN token rows, persistent over the tiles.
__global__ void __launch_bounds__(kHeadThreads, 1) head_proj_kernel(const __grid_constant__ CUtensorMap map_w,
                                                                    const __grid_constant__ CUtensorMap map_x,
                                                                    const HeadParams P)
{
    extern __shared__ uint8_t smem_raw[];
    uint8_t *smem = reinterpret_cast<uint8_t *>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
    uint64_t *full_bar = reinterpret_cast<uint64_t *>(smem + static_cast<size_t>(P.stages) * P.stage_bytes);
    uint64_t *empty_bar = full_bar + kMaxStages;
    uint64_t *acc_full = empty_bar + kMaxStages;  // [2]
    uint64_t *acc_empty = acc_full + 2;           // [2]
    uint32_t *tmem_slot = reinterpret_cast<uint32_t *>(acc_empty + 2);
    volatile int *abort_flag = reinterpret_cast<volatile int *>(tmem_slot + 1);

    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    hawk::allow_dependent_launch();
    const int kblocks = P.hidden / kBK;
    const int total_tiles = P.tiles_m * P.tiles_n;

    if (tid == 0) {
        for (int i = 0; i < P.stages; ++i) {
            mbar_init(&full_bar[i], 1);
            mbar_init(&empty_bar[i], 1);
        }
        for (int i = 0; i < 2; ++i) {
            mbar_init(&acc_full[i], 1);
            mbar_init(&acc_empty[i], 4);  // one arrival per epilogue warp
        }
        *abort_flag = 0;
        fence_mbar_init();
    }
    if (warp == 1) {
        tmem_alloc(tmem_slot, kTmemCols);
        tmem_relinquish();
    }
    tcgen05_fence_before();
    __syncthreads();
    tcgen05_fence_after();
    const uint32_t tmem_base = *tmem_slot;
    grid_dependency_wait();  // set-up above overlaps the previous kernel; global memory is touched from here on

    if (warp == 0) {
        // =========================== TMA producer
        if (lane == 0) {
            prefetch_tensormap(&map_w);
            prefetch_tensormap(&map_x);
            const uint32_t tx_bytes = static_cast<uint32_t>(P.stage_bytes);
            int st = 0;
            uint32_t ph = 0;
            bool ok = true;
            long long issued = 0;
            for (int tile = blockIdx.x; tile < total_tiles && ok; tile += gridDim.x) {
                const int tn = tile % P.tiles_n, tm = tile / P.tiles_n;
                const int row_w = P.v_begin + tm * kBM, row_x = tn * P.BN;
                for (int kb = 0; kb < kblocks; ++kb) {
                    ok = mbar_wait(&empty_bar[st], ph ^ 1u, abort_flag);
                    if (!ok) break;
                    uint8_t *a = smem + static_cast<size_t>(st) * P.stage_bytes;
                    // (test builds only: the first stage of block 0 is armed for more bytes than arrive)
                    const bool stall = kTestStallBytes != 0 && blockIdx.x == 0 && issued == 0;
                    mbar_arrive_expect_tx(&full_bar[st], tx_bytes + (stall ? kTestStallBytes : 0u));
                    tma_load_2d(a, &map_w, kb * kBK, row_w, &full_bar[st]);
                    if (P.pairs == 0) {
                        tma_load_2d(a + kATileBytes, &map_x, kb * kBK, row_x, &full_bar[st]);
                    } else {  // conditional rows of the tile's pairs, then their unconditional rows
                        const int half = P.BN / 2;
                        tma_load_2d(a + kATileBytes, &map_x, kb * kBK, tn * half, &full_bar[st]);
                        tma_load_2d(a + kATileBytes + half * kBK * 2, &map_x, kb * kBK, P.pairs + tn * half,
                                    &full_bar[st]);
                    }
                    ++issued;
                    if (++st == P.stages) {
                        st = 0;
                        ph ^= 1u;
                    }
                }
            }
            if (!ok) {
                *abort_flag = 1;
                if (P.dev_status) atomicOr(P.dev_status, HAWK_DEV_TIMEOUT);
            }
        }
    } else if (warp == 1) {
        // =========================== MMA issuer
        if (lane == 0) {
            const uint32_t idesc = umma_idesc_bf16_f32(kBM, P.BN);
            int st = 0;
            uint32_t ph = 0;
            bool ok = true;
            int it = 0;
            for (int tile = blockIdx.x; tile < total_tiles && ok; tile += gridDim.x, ++it) {
                const int ab = it & 1;
                const uint32_t acc_ph = (it >> 1) & 1;
                ok = mbar_wait(&acc_empty[ab], acc_ph ^ 1u, abort_flag);  // epilogue drained this buffer
                if (!ok) break;
                tcgen05_fence_after();
                const uint32_t d_tmem = tmem_base + static_cast<uint32_t>(ab * P.BN);
                for (int kb = 0; kb < kblocks; ++kb) {
                    ok = mbar_wait(&full_bar[st], ph, abort_flag);
                    if (!ok) break;
                    tcgen05_fence_after();
                    const uint32_t a_addr = smem_u32(smem + static_cast<size_t>(st) * P.stage_bytes);
                    const uint64_t da = umma_desc_k_major_sw128(a_addr);
                    const uint64_t db = umma_desc_k_major_sw128(a_addr + kATileBytes);
#pragma unroll
                    for (int k = 0; k < kBK / 16; ++k) {
                        // 16 bf16 along K = 32 bytes = 2 units of the descriptor's 16-byte address field
                        umma_bf16(d_tmem, da + static_cast<uint64_t>(2 * k), db + static_cast<uint64_t>(2 * k), idesc,
                                  (kb | k) != 0 ? 1u : 0u);
                    }
                    umma_commit(&empty_bar[st]);  // stage reusable once these MMAs have read it
                    if (++st == P.stages) {
                        st = 0;
                        ph ^= 1u;
                    }
                }
                if (!ok) break;
                umma_commit(&acc_full[ab]);  // accumulator complete
            }
            if (!ok) {
                *abort_flag = 1;
                if (P.dev_status) atomicOr(P.dev_status, HAWK_DEV_TIMEOUT);
            }
        }
    } else {
        // =========================== epilogue warps: TMEM lanes 32*(warp%4) .. +31
        const int lane_base = (warp & 3) * 32;
        bool ok = true;
        int it = 0;
        for (int tile = blockIdx.x; tile < total_tiles && ok; tile += gridDim.x, ++it) {
            const int tn = tile % P.tiles_n, tm = tile / P.tiles_n;
            const int ab = it & 1;
            const uint32_t acc_ph = (it >> 1) & 1;
            ok = mbar_wait(&acc_full[ab], acc_ph, abort_flag);
            if (!ok) break;
            tcgen05_fence_after();
            const int v = P.v_begin + tm * kBM + lane_base + lane;  // this thread's token id
            const bool v_ok = v < P.v_end;
            const uint32_t taddr = tmem_base + (static_cast<uint32_t>(lane_base) << 16) + static_cast<uint32_t>(ab * P.BN);
            epilogue_store(P, taddr, tn, v, v_ok);
            tcgen05_fence_before();
            __syncwarp();
            if (lane == 0) mbar_arrive(&acc_empty[ab]);
        }
        if (!ok && lane == 0) {
            *abort_flag = 1;
            if (P.dev_status) atomicOr(P.dev_status, HAWK_DEV_TIMEOUT);
        }
    }

    tcgen05_fence_before();
    __syncthreads();
    if (warp == 1) {
        tcgen05_fence_after();
        tmem_dealloc(tmem_base, kTmemCols);
    }
}



// Few tiles and a long hidden dimension: launched as clusters of two blocks, one tile per cluster: block r multiplies over half r of the hidden
// dimension; the blocks then swap halves of their accumulators through distributed shared memory (16-column chunks
// alternate between them), each adds its partner's sums to its own for the chunks it owns (one addition of two
// numbers: the result does not depend on timing or on which block does it), applies the guidance combine if asked to,
// and stores.  No zeroed output, no atomics, and the plain and the guided form sum in the same way.
__global__ void __launch_bounds__(kHeadThreads, 1) head_proj_split_kernel(const __grid_constant__ CUtensorMap map_w,
                                                                    const __grid_constant__ CUtensorMap map_x,
                                                                    const HeadParams P)
{
    extern __shared__ uint8_t smem_raw[];
    uint8_t *smem = reinterpret_cast<uint8_t *>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
    uint64_t *full_bar = reinterpret_cast<uint64_t *>(smem + static_cast<size_t>(P.stages) * P.stage_bytes);
    uint64_t *empty_bar = full_bar + kMaxStages;
    uint64_t *acc_full = empty_bar + kMaxStages;  // [2]
    uint64_t *acc_empty = acc_full + 2;           // [2]
    uint32_t *tmem_slot = reinterpret_cast<uint32_t *>(acc_empty + 2);
    volatile int *abort_flag = reinterpret_cast<volatile int *>(tmem_slot + 1);

    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    hawk::allow_dependent_launch();
    const int kblocks = P.hidden / kBK;
    // a block's unit of work is the half of its pair's tile that its rank in the pair names (the launch gives every
    // pair exactly one tile; the loops below are written like the unsplit kernel's and run once)
    const int total_tiles = P.tiles_m * P.tiles_n;
    const int kb_half = (kblocks + 1) / 2;
    const int part = static_cast<int>(cluster_cta_rank());
    const int first_tile = static_cast<int>(blockIdx.x >> 1);
    const int tile_step = static_cast<int>(gridDim.x >> 1);

    if (tid == 0) {
        for (int i = 0; i < P.stages; ++i) {
            mbar_init(&full_bar[i], 1);
            mbar_init(&empty_bar[i], 1);
        }
        for (int i = 0; i < 2; ++i) {
            mbar_init(&acc_full[i], 1);
            mbar_init(&acc_empty[i], 4);  // one arrival per epilogue warp
        }
        *abort_flag = 0;
        fence_mbar_init();
    }
    if (warp == 1) {
        tmem_alloc(tmem_slot, kTmemCols);
        tmem_relinquish();
    }
    tcgen05_fence_before();
    __syncthreads();
    tcgen05_fence_after();
    const uint32_t tmem_base = *tmem_slot;
    grid_dependency_wait();  // set-up above overlaps the previous kernel; global memory is touched from here on

    if (warp == 0) {
        // =========================== TMA producer
        if (lane == 0) {
            prefetch_tensormap(&map_w);
            prefetch_tensormap(&map_x);
            const uint32_t tx_bytes = static_cast<uint32_t>(P.stage_bytes);
            int st = 0;
            uint32_t ph = 0;
            bool ok = true;
            long long issued = 0;
            for (int tile = first_tile; tile < total_tiles && ok; tile += tile_step) {
                const int tn = tile % P.tiles_n, tm = tile / P.tiles_n;
                const int row_w = P.v_begin + tm * kBM, row_x = tn * P.BN;
                const int kb0 = part * kb_half, kb1 = min(kblocks, kb0 + kb_half);
                for (int kb = kb0; kb < kb1; ++kb) {
                    ok = mbar_wait(&empty_bar[st], ph ^ 1u, abort_flag);
                    if (!ok) break;
                    uint8_t *a = smem + static_cast<size_t>(st) * P.stage_bytes;
                    // (test builds only: the first stage of block 0 is armed for more bytes than arrive)
                    const bool stall = kTestStallBytes != 0 && blockIdx.x == 0 && issued == 0;
                    mbar_arrive_expect_tx(&full_bar[st], tx_bytes + (stall ? kTestStallBytes : 0u));
                    tma_load_2d(a, &map_w, kb * kBK, row_w, &full_bar[st]);
                    if (P.pairs == 0) {
                        tma_load_2d(a + kATileBytes, &map_x, kb * kBK, row_x, &full_bar[st]);
                    } else {  // conditional rows of the tile's pairs, then their unconditional rows
                        const int half = P.BN / 2;
                        tma_load_2d(a + kATileBytes, &map_x, kb * kBK, tn * half, &full_bar[st]);
                        tma_load_2d(a + kATileBytes + half * kBK * 2, &map_x, kb * kBK, P.pairs + tn * half,
                                    &full_bar[st]);
                    }
                    ++issued;
                    if (++st == P.stages) {
                        st = 0;
                        ph ^= 1u;
                    }
                }
            }
            if (!ok) {
                *abort_flag = 1;
                if (P.dev_status) atomicOr(P.dev_status, HAWK_DEV_TIMEOUT);
            }
        }
    } else if (warp == 1) {
        // =========================== MMA issuer
        if (lane == 0) {
            const uint32_t idesc = umma_idesc_bf16_f32(kBM, P.BN);
            int st = 0;
            uint32_t ph = 0;
            bool ok = true;
            int it = 0;
            for (int tile = first_tile; tile < total_tiles && ok; tile += tile_step, ++it) {
                const int ab = it & 1;
                const uint32_t acc_ph = (it >> 1) & 1;
                ok = mbar_wait(&acc_empty[ab], acc_ph ^ 1u, abort_flag);  // epilogue drained this buffer
                if (!ok) break;
                tcgen05_fence_after();
                const uint32_t d_tmem = tmem_base + static_cast<uint32_t>(ab * P.BN);
                const int kb0 = part * kb_half, kb1 = min(kblocks, kb0 + kb_half);
                for (int kb = kb0; kb < kb1; ++kb) {
                    ok = mbar_wait(&full_bar[st], ph, abort_flag);
                    if (!ok) break;
                    tcgen05_fence_after();
                    const uint32_t a_addr = smem_u32(smem + static_cast<size_t>(st) * P.stage_bytes);
                    const uint64_t da = umma_desc_k_major_sw128(a_addr);
                    const uint64_t db = umma_desc_k_major_sw128(a_addr + kATileBytes);
#pragma unroll
                    for (int k = 0; k < kBK / 16; ++k) {
                        // 16 bf16 along K = 32 bytes = 2 units of the descriptor's 16-byte address field
                        umma_bf16(d_tmem, da + static_cast<uint64_t>(2 * k), db + static_cast<uint64_t>(2 * k), idesc,
                                  ((kb - kb0) | k) != 0 ? 1u : 0u);
                    }
                    umma_commit(&empty_bar[st]);  // stage reusable once these MMAs have read it
                    if (++st == P.stages) {
                        st = 0;
                        ph ^= 1u;
                    }
                }
                if (!ok) break;
                umma_commit(&acc_full[ab]);  // accumulator complete
            }
            if (!ok) {
                *abort_flag = 1;
                if (P.dev_status) atomicOr(P.dev_status, HAWK_DEV_TIMEOUT);
            }
        }
    } else {
        // =========================== epilogue warps: TMEM lanes 32*(warp%4) .. +31
        const int lane_base = (warp & 3) * 32;
        bool ok = true;
        int it = 0;
        for (int tile = first_tile; tile < total_tiles && ok; tile += tile_step, ++it) {
            const int tn = tile % P.tiles_n, tm = tile / P.tiles_n;
            const int ab = it & 1;
            const uint32_t acc_ph = (it >> 1) & 1;
            ok = mbar_wait(&acc_full[ab], acc_ph, abort_flag);
            if (!ok) break;
            tcgen05_fence_after();
            const int v = P.v_begin + tm * kBM + lane_base + lane;  // this thread's token id
            const bool v_ok = v < P.v_end;
            const uint32_t taddr = tmem_base + (static_cast<uint32_t>(lane_base) << 16) + static_cast<uint32_t>(ab * P.BN);
            // each block hands the other the chunks that one will finish; the stores follow once the pair has met
            (void)tn, (void)v_ok;
            epilogue_send(P, taddr, lane_base + lane, map_shared_to_cta(smem + P.xchg_off, part ^ 1), part ^ 1);
            tcgen05_fence_before();
            __syncwarp();
            if (lane == 0) mbar_arrive(&acc_empty[ab]);
        }
        if (!ok && lane == 0) {
            *abort_flag = 1;
            if (P.dev_status) atomicOr(P.dev_status, HAWK_DEV_TIMEOUT);
        }
    }

    tcgen05_fence_before();
    __syncthreads();
    {
        // every thread of both blocks gets here, whatever happened above: each block now holds its partner's sums for
        // the chunks it owns
        cluster_sync_all();
        if (warp >= 2 && first_tile < total_tiles && !*abort_flag) {
            tcgen05_fence_after();
            const int lane_base = (warp & 3) * 32;
            const int tn = first_tile % P.tiles_n, tm = first_tile / P.tiles_n;
            const int v = P.v_begin + tm * kBM + lane_base + lane;
            const uint32_t taddr = tmem_base + (static_cast<uint32_t>(lane_base) << 16);
            epilogue_store<true>(P, taddr, tn, v, v < P.v_end, part, 2, reinterpret_cast<const float *>(smem + P.xchg_off),
                                 lane_base + lane);
            tcgen05_fence_before();
        }
        __syncthreads();
    }
    if (warp == 1) {
        tcgen05_fence_after();
        tmem_dealloc(tmem_base, kTmemCols);
    }
}


// ------------------------------------------------------------------------------------------------
// The same projection by pairs of CTAs (clusters of two) that drive one MMA of 256 token ids x BN
// token rows together (tcgen05 cta_group::2).  Each CTA of a pair loads its own 128 weight rows and
// only HALF of the tile's token rows; the tensor cores of both SMs read both halves.  Per flop a CTA
// moves two thirds of the shared-memory bytes of the single-CTA kernel (fills and operand reads), which
// is what bounds that kernel once there are enough token rows to be tensor-bound.
//   warp 0      TMA producer (own weight rows, own half of the token rows), in both CTAs
//   warp 1      rank 0: issues the pair MMAs and commits to the barriers of both CTAs
//               (both CTAs' loads count on rank 0's stage barrier)
//   warps 2..9  epilogue of the CTA's own 128 accumulator rows, in both CTAs: two warps per lane
//               quarter, taking alternate 16-column chunks
// Tensor memory is allocated and freed by warp 1 of each CTA of the pair.
#ifndef HAWK_PAIR_TMEM_COLS
#define HAWK_PAIR_TMEM_COLS 512
#endif
constexpr uint32_t kPairTmemCols = HAWK_PAIR_TMEM_COLS;

constexpr int kPairThreads = 320;  // producer, MMA, and two epilogue warps per tensor-memory lane quarter

template <bool WIDE>
__global__ void __cluster_dims__(2, 1, 1) __launch_bounds__(kPairThreads, 1)
    head_proj_pair_kernel(const __grid_constant__ CUtensorMap map_w, const __grid_constant__ CUtensorMap map_x,
                          const HeadParams P)
{
    extern __shared__ uint8_t smem_raw[];
    uint8_t *smem = reinterpret_cast<uint8_t *>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
    uint64_t *full_bar = reinterpret_cast<uint64_t *>(smem + static_cast<size_t>(P.stages) * P.stage_bytes);
    uint64_t *empty_bar = full_bar + kMaxStages;
    uint64_t *acc_full = empty_bar + kMaxStages;   // [2]
    uint64_t *acc_empty = acc_full + 2;            // [2], used in rank 0: 4 epilogue warps of each CTA
    uint32_t *tmem_slot = reinterpret_cast<uint32_t *>(acc_empty + 2);
    volatile int *abort_flag = reinterpret_cast<volatile int *>(tmem_slot + 1);

    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    const uint32_t rank = cluster_cta_rank();
    const int pair = blockIdx.x >> 1, n_pairs = gridDim.x >> 1;
    hawk::allow_dependent_launch();
    const int kblocks = P.hidden / kBK;
    const int total_tiles = P.tiles_m * P.tiles_n;
    const int half_n = P.BN / 2;

    if (tid == 0) {
        for (int i = 0; i < P.stages; ++i) {
            mbar_init(&full_bar[i], 1);
            mbar_init(&empty_bar[i], 1);
        }
        for (int i = 0; i < 2; ++i) {
            mbar_init(&acc_full[i], 1);
            mbar_init(&acc_empty[i], 16);  // 8 epilogue warps in each CTA
        }
        *abort_flag = 0;
        fence_mbar_init();
    }
    if (warp == 1) {
        tmem_alloc_pair(tmem_slot, kPairTmemCols);
        tmem_relinquish_pair();
    }
    tcgen05_fence_before();
    __syncthreads();
    cluster_sync_all();  // the other CTA's barriers exist before anything is signalled across
    tcgen05_fence_after();
    const uint32_t tmem_base = *tmem_slot;
    grid_dependency_wait();

    if (warp == 0) {
        // =========================== TMA producer (both CTAs)
        if (lane == 0) {
            prefetch_tensormap(&map_w);
            prefetch_tensormap(&map_x);
            const uint32_t tx_bytes = static_cast<uint32_t>(P.stage_bytes);
            int st = 0;
            uint32_t ph = 0;
            bool ok = true;
            for (int tile = pair; tile < total_tiles && ok; tile += n_pairs) {
                const int tn = tile % P.tiles_n, tm = tile / P.tiles_n;
                const int row_w = P.v_begin + tm * (2 * kBM) + static_cast<int>(rank) * kBM;
                const int row_x = P.pairs == 0 ? tn * P.BN + static_cast<int>(rank) * half_n
                                               : (rank == 0 ? tn * half_n : P.pairs + tn * half_n);
                for (int kb = 0; kb < kblocks; ++kb) {
                    ok = mbar_wait_cluster(&empty_bar[st], ph ^ 1u, abort_flag);
                    if (!ok) break;
                    uint8_t *a = smem + static_cast<size_t>(st) * P.stage_bytes;
                    // (test builds only: the first stage of pair 0 is armed for more bytes than arrive)
                    const bool stall = kTestStallBytes != 0 && pair == 0 && tile == pair && kb == 0;
                    if (rank == 0) mbar_arrive_expect_tx(&full_bar[st], 2 * tx_bytes + (stall ? kTestStallBytes : 0u));  // both CTAs' halves
                    const uint32_t bar0 = map_shared_to_cta(&full_bar[st], 0);
                    tma_load_2d_pair(a, &map_w, kb * kBK, row_w, bar0);
                    tma_load_2d_pair(a + kATileBytes, &map_x, kb * kBK, row_x, bar0);
                    if (++st == P.stages) {
                        st = 0;
                        ph ^= 1u;
                    }
                }
            }
            if (!ok) {
                *abort_flag = 1;
                if (P.dev_status) atomicOr(P.dev_status, HAWK_DEV_TIMEOUT);
            }
        }
    } else if (warp == 1 && rank != 0) {
        // rank 1's warp 1 only allocates and frees tensor memory
    } else if (warp == 1) {
        // =========================== rank 0: MMA issuer for the pair
        if (lane == 0) {
            const int mma_n = WIDE ? P.BN / 2 : P.BN;  // columns per MMA
            const uint32_t idesc = umma_idesc_bf16_f32(2 * kBM, mma_n);
            int st = 0;
            uint32_t ph = 0;
            bool ok = true;
            int it = 0;
            for (int tile = pair; tile < total_tiles && ok; tile += n_pairs, ++it) {
                const int ab = WIDE ? 0 : it & 1;  // WIDE: one accumulator fills tensor memory
                const uint32_t acc_ph = WIDE ? it & 1 : (it >> 1) & 1;
                ok = mbar_wait_cluster(&acc_empty[ab], acc_ph ^ 1u, abort_flag);  // both epilogues drained it
                if (!ok) break;
                tcgen05_fence_after();
                const uint32_t d_tmem = tmem_base + static_cast<uint32_t>(ab * P.BN);
                for (int kb = 0; kb < kblocks; ++kb) {
                    ok = mbar_wait_cluster(&full_bar[st], ph, abort_flag);  // both CTAs' halves have landed
                    if (!ok) break;
                    tcgen05_fence_after();
                    const uint32_t a_addr = smem_u32(smem + static_cast<size_t>(st) * P.stage_bytes);
                    const uint64_t da = umma_desc_k_major_sw128(a_addr);
                    const uint64_t db = umma_desc_k_major_sw128(a_addr + kATileBytes);
#pragma unroll
                    for (int k = 0; k < kBK / 16; ++k) {
                        umma_bf16_pair(d_tmem, da + static_cast<uint64_t>(2 * k), db + static_cast<uint64_t>(2 * k), idesc,
                                       (kb | k) != 0 ? 1u : 0u);
                        if constexpr (WIDE) {  // second half of the columns: rows BN / 4 onwards of each CTA's token rows
                            const uint64_t db2 = umma_desc_k_major_sw128(a_addr + kATileBytes + (P.BN / 4) * kBK * 2);
                            umma_bf16_pair(d_tmem + static_cast<uint32_t>(mma_n), da + static_cast<uint64_t>(2 * k),
                                           db2 + static_cast<uint64_t>(2 * k), idesc, (kb | k) != 0 ? 1u : 0u);
                        }
                    }
                    umma_commit_pair(&empty_bar[st], 3);  // the stage is reusable in both CTAs
                    if (++st == P.stages) {
                        st = 0;
                        ph ^= 1u;
                    }
                }
                if (!ok) break;
                umma_commit_pair(&acc_full[ab], 3);  // accumulator complete, in both CTAs
            }
            if (!ok) {
                *abort_flag = 1;
                if (P.dev_status) atomicOr(P.dev_status, HAWK_DEV_TIMEOUT);
            }
        }
    } else {
        // =========================== epilogue warps (both CTAs): own TMEM lanes 32*(warp%4) .. +31
        const int lane_base = (warp & 3) * 32;
        const uint32_t acc_empty_rank0[2] = {map_shared_to_cta(&acc_empty[0], 0), map_shared_to_cta(&acc_empty[1], 0)};
        bool ok = true;
        int it = 0;
        for (int tile = pair; tile < total_tiles && ok; tile += n_pairs, ++it) {
            const int tn = tile % P.tiles_n, tm = tile / P.tiles_n;
            const int ab = WIDE ? 0 : it & 1;
            const uint32_t acc_ph = WIDE ? it & 1 : (it >> 1) & 1;
            ok = mbar_wait_cluster(&acc_full[ab], acc_ph, abort_flag);
            if (!ok) break;
            tcgen05_fence_after();
            const int v = P.v_begin + tm * (2 * kBM) + static_cast<int>(rank) * kBM + lane_base + lane;
            const bool v_ok = v < P.v_end;
            const uint32_t taddr = tmem_base + (static_cast<uint32_t>(lane_base) << 16) + static_cast<uint32_t>(ab * P.BN);
            epilogue_store<false, WIDE>(P, taddr, tn, v, v_ok, (warp - 2) >> 2, 2);
            tcgen05_fence_before();
            __syncwarp();
            if (lane == 0) mbar_arrive_cluster(acc_empty_rank0[ab]);
        }
        if (!ok && lane == 0) {
            *abort_flag = 1;
            if (P.dev_status) atomicOr(P.dev_status, HAWK_DEV_TIMEOUT);
        }
    }

    tcgen05_fence_before();
    __syncthreads();
    cluster_sync_all();  // neither CTA frees tensor memory or exits while the other may still use or signal it
    if (warp == 1) {
        tcgen05_fence_after();
        tmem_dealloc_pair(tmem_base, kPairTmemCols);
    }
}


}  // namespace

hawk_status hawk_host::check_head_proj_args(const void *x, const void *w, const float *logits, int M, int hidden, int V,
                                            int v_begin, int v_end)
{
    if (M < 0 || hidden < 0 || V < 0) return HAWK_ERR_SHAPE;
    if (v_begin < 0 || v_end > V || v_begin > v_end) return HAWK_ERR_SHAPE;
    if (M == 0 || v_begin == v_end) return HAWK_OK;
    if (!x || !w || !logits) return HAWK_ERR_NULL;
    if (hidden < 64 || hidden % 64 != 0) return HAWK_ERR_UNSUPPORTED;
    if (!hawk_host::aligned16(x) || !hawk_host::aligned16(w) || !hawk_host::aligned16(logits)) return HAWK_ERR_ALIGN;
    return HAWK_OK;
}

namespace {
// pairs == 0: logits [M][V]; pairs > 0: M == 2 * pairs and `logits` receives guided rows [pairs][V].
hawk_status head_proj_impl(const void *x, const void *w, float *logits, int M, int pairs, float cfg_scale,
                           float temperature, int hidden, int V, int v_begin, int v_end, int32_t *dev_status,
                           hawk_stream_t stream)
{
    const hawk_status chk = hawk_host::check_head_proj_args(x, w, logits, M, hidden, V, v_begin, v_end);
    if (chk != HAWK_OK) return chk;
    if (M == 0 || v_begin == v_end) return HAWK_OK;
    int sm_count = 0;
    if (!hawk_host::is_sm100(&sm_count)) return HAWK_ERR_UNSUPPORTED;

    HeadParams P;
    P.logits = logits;
    P.M = M;
    P.hidden = hidden;
    P.V = V;
    P.v_begin = v_begin;
    P.v_end = v_end;
    P.pairs = pairs;
    P.cfg_scale = cfg_scale;
    P.temperature = temperature;
    // From HAWK_HEAD_PAIR_MIN_ROWS token rows on, pairs of CTAs share a tile (cta_group::2).  Measured: with
    // 1024 rows the pair kernel takes 42 us where the single-CTA kernel takes 45; with 384 rows they tie; below
    // that the call is bound by the weight stream and the single-CTA kernel, with twice as many tiles, is ahead.
#ifndef HAWK_HEAD_PAIR_MIN_ROWS
#define HAWK_HEAD_PAIR_MIN_ROWS 512
#endif
    // Between 257 and 511 token rows the pair kernel takes all rows as ONE tile of up to 512 columns (one
    // accumulator, no overlap of epilogue and MMAs, but a single round of tiles whose MMAs are wide enough to hide
    // their issue cost): 25.6 -> measured below at 384 rows.
    const bool wide = M > 256 && M < HAWK_HEAD_PAIR_MIN_ROWS && sm_count >= 2 && kPairTmemCols == 512;
    const bool use_pair = (M >= HAWK_HEAD_PAIR_MIN_ROWS || wide) && sm_count >= 2;
    const int max_bn = wide ? 512 : use_pair ? static_cast<int>(kPairTmemCols) / 2 : 256;  // accumulators in tensor memory
    const int bn_step = wide ? 64 : use_pair ? 32 : 16;  // a pair's tile splits into halves of a multiple of 16 rows
    P.wide = wide ? 1 : 0;
    int x_box_rows;
    if (pairs == 0) {
        P.tiles_n = (M + max_bn - 1) / max_bn;
        const int per_tile = (M + P.tiles_n - 1) / P.tiles_n;
        P.BN = (per_tile + bn_step - 1) / bn_step * bn_step;
        x_box_rows = use_pair ? P.BN / 2 : P.BN;
    } else {  // half a tile of conditional rows, half of unconditional ones; each half a multiple of 16 (32 when wide)
        P.tiles_n = (pairs + max_bn / 2 - 1) / (max_bn / 2);
        const int per_tile = (pairs + P.tiles_n - 1) / P.tiles_n;
        const int step = wide ? 32 : 16;
        x_box_rows = (per_tile + step - 1) / step * step;
        P.BN = 2 * x_box_rows;
    }
    const int tile_rows = use_pair ? 2 * kBM : kBM;  // token ids per tile
    P.tiles_m = (v_end - v_begin + tile_rows - 1) / tile_rows;
    P.stage_bytes = kATileBytes + x_box_rows * kBK * 2 * (pairs != 0 && !use_pair ? 2 : 1);
    // few tiles and a long hidden dimension (a narrow valid range of a wide model): a pair of blocks per tile, each
    // over half of the hidden dimension, so that twice as many SMs stream the weights
    P.ksplit = (!use_pair && 2 * P.tiles_m * P.tiles_n <= sm_count && hidden / kBK >= 16) ? 2 : 1;
    const int xchg_bytes = P.ksplit > 1 ? kBM * P.BN * 4 : 0;  // block 1's sums, received by block 0
    const int smem_budget = 200 * 1024 - xchg_bytes;
    int stages = smem_budget / P.stage_bytes;
    if (stages > kMaxStages) stages = kMaxStages;
    if (stages < 2) return HAWK_ERR_UNSUPPORTED;
    P.stages = stages;
    P.dev_status = dev_status;

    CUtensorMap map_w, map_x;
    if (!hawk_host::encode_bf16_rows_sw128(&map_w, w, static_cast<uint64_t>(V), static_cast<uint64_t>(hidden), kBM,
                                           true) ||
        !hawk_host::encode_bf16_rows_sw128(&map_x, x, static_cast<uint64_t>(M), static_cast<uint64_t>(hidden),
                                           static_cast<uint32_t>(x_box_rows), true))
        return HAWK_ERR_CUDA;

    // always ask for enough shared memory that a second block cannot share the SM: each block owns all of TMEM
    P.xchg_off = ((stages * P.stage_bytes + (3 * kMaxStages + 4) * 8 + 64 + 1023) / 1024) * 1024;
    const size_t smem_bytes = 1024 + static_cast<size_t>(P.xchg_off) + xchg_bytes;
    const size_t smem_req = smem_bytes < 120 * 1024 ? 120 * 1024 : smem_bytes;
    int device = 0;
    if (cudaGetDevice(&device) != cudaSuccess || device < 0 || device >= 64) return HAWK_ERR_CUDA;
    static std::atomic<unsigned long long> attr_done{0};  // per device: the dynamic shared memory limit is a per-device attribute
    if (!((attr_done.load(std::memory_order_relaxed) >> device) & 1ull)) {
        if (cudaFuncSetAttribute(head_proj_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, 227 * 1024) !=
                cudaSuccess ||
            cudaFuncSetAttribute(head_proj_split_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, 227 * 1024) !=
                cudaSuccess ||
            cudaFuncSetAttribute(head_proj_pair_kernel<false>, cudaFuncAttributeMaxDynamicSharedMemorySize, 227 * 1024) !=
                cudaSuccess ||
            cudaFuncSetAttribute(head_proj_pair_kernel<true>, cudaFuncAttributeMaxDynamicSharedMemorySize, 227 * 1024) !=
                cudaSuccess)
            return HAWK_ERR_CUDA;
        attr_done.fetch_or(1ull << device, std::memory_order_relaxed);
    }
    const int total_tiles = P.tiles_m * P.tiles_n;
    cudaError_t err;
    if (use_pair) {
        // pairs that can be resident at once (an SM without a free neighbour in its group takes none): a
        // persistent grid larger than that would run its last pairs after all the others have finished
        static std::atomic<int> max_pairs_of[64];  // per device, looked up once (two threads may both look it up: same value)
        int max_pairs = max_pairs_of[device].load(std::memory_order_relaxed);
        if (max_pairs == 0) {
            cudaLaunchConfig_t occ = {};
            occ.gridDim = dim3(sm_count / 2 * 2);
            occ.blockDim = dim3(kPairThreads);
            occ.dynamicSmemBytes = 227 * 1024 - 1024;
            int n = 0;
            if (cudaOccupancyMaxActiveClusters(&n, head_proj_pair_kernel<false>, &occ) != cudaSuccess || n < 1) {
                (void)cudaGetLastError();
                n = sm_count / 4;  // conservative: half of the SMs
            }
            max_pairs = n < sm_count / 2 ? n : sm_count / 2;
            max_pairs_of[device].store(max_pairs, std::memory_order_relaxed);
        }
        const int n_pairs = total_tiles < max_pairs ? total_tiles : max_pairs;
        err = hawk_host::launch_dependent(wide ? head_proj_pair_kernel<true> : head_proj_pair_kernel<false>,
                                          dim3(2 * n_pairs), dim3(kPairThreads), smem_req,
                                          reinterpret_cast<cudaStream_t>(stream), map_w, map_x, P);
    } else {
        if (P.ksplit > 1) {  // one cluster of two blocks per tile
            cudaLaunchAttribute attr[2];
            attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
            attr[0].val.programmaticStreamSerializationAllowed = 1;
            attr[1].id = cudaLaunchAttributeClusterDimension;
            attr[1].val.clusterDim.x = 2;
            attr[1].val.clusterDim.y = 1;
            attr[1].val.clusterDim.z = 1;
            cudaLaunchConfig_t cfg = {};
            cfg.gridDim = dim3(2 * total_tiles);
            cfg.blockDim = dim3(kHeadThreads);
            cfg.dynamicSmemBytes = smem_req;
            cfg.stream = reinterpret_cast<cudaStream_t>(stream);
            cfg.attrs = attr;
            cfg.numAttrs = 2;
            err = cudaLaunchKernelEx(&cfg, head_proj_split_kernel, map_w, map_x, P);
        } else {
            const int grid = total_tiles < sm_count ? total_tiles : sm_count;
            err = hawk_host::launch_dependent(head_proj_kernel, dim3(grid), dim3(kHeadThreads), smem_req,
                                              reinterpret_cast<cudaStream_t>(stream), map_w, map_x, P);
        }
    }
    return err == cudaSuccess ? HAWK_OK : HAWK_ERR_CUDA;
}
}  // namespace

extern "C" hawk_status hawk_head_proj(const void *x, const void *w, float *logits, int M, int hidden, int V,
                                      int v_begin, int v_end, int32_t *dev_status, hawk_stream_t stream)
{
    const hawk_host::NvtxRange nvtx_range("hawk_head_proj");
    return head_proj_impl(x, w, logits, M, 0, 1.0f, 1.0f, hidden, V, v_begin, v_end, dev_status, stream);
}

extern "C" hawk_status hawk_head_proj_cfg(const void *x, const void *w, float *guided, int B, int rows, int hidden,
                                          int V, int v_begin, int v_end, float cfg_scale, float temperature,
                                          int32_t *dev_status, hawk_stream_t stream)
{
    const hawk_host::NvtxRange nvtx_range("hawk_head_proj_cfg");
    if (B < 0 || rows < 0) return HAWK_ERR_SHAPE;
    if (static_cast<long long>(B) * rows > (1 << 29)) return HAWK_ERR_UNSUPPORTED;
    if (!(temperature == temperature) || !(cfg_scale == cfg_scale) || isinf(temperature) || isinf(cfg_scale) ||
        !(temperature > 0.f))
        return HAWK_ERR_PARAM;
    const int pairs = B * rows;
    return head_proj_impl(x, w, guided, 2 * pairs, pairs, cfg_scale, temperature, hidden, V, v_begin, v_end, dev_status,
                          stream);
}
