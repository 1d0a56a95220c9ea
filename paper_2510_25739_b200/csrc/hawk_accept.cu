// hawk_cfg_accept: guidance combine, temperature, top-k, softmax, acceptance test and residual
// resampling.
//
// One thread block per (sequence, draft position) row.  The row of guided logits lives in registers
// from the moment it is read (each logit row is read from HBM exactly once); the target
// probabilities p and the residual max(0, p - q) are never written back.  Draft probabilities q are
// read only by rows whose draft was rejected.  A second, tiny kernel picks, per sequence, the first
// rejected row.
// The kernel is a chain of short block-wide phases (range, histogram select, softmax sum, scan), so
// what bounds it is the length of that chain: the block is as wide as the row allows (16 ids per
// thread, up to 1024 threads) and every phase is a handful of instructions per thread.
// (Splitting a row over a cluster of blocks was measured: each cluster-wide exchange costs about
// 1.2 us, five of them per row cost more than the wider load path saves.)
//
// Rule implemented: accept draft x iff u * q(x) < p(x); at the first rejection draw the
// correction token from norm(max(0, p - q)) by inverse CDF in ascending token id
// (speculative sampling, Sec. 3; chain verification and residual update, Sec. 4.2).
#include <math_constants.h>

#include <mutex>

#include <climits>

#include "hawk_common.cuh"

namespace {

constexpr int kBins = 1024;     // histogram bins of one top-k selection round
constexpr int kCandMax = 1024;  // members of the selected bin that are ranked exactly in shared memory
constexpr int kMaxRounds = 48;  // each narrowing round shrinks the value range by >= 1024x; fp32 allows < 8

constexpr int ROW_ACCEPTED = -1;
constexpr int ROW_REJECTED_NO_TOKEN = -2;  // rejected and nothing has positive mass
constexpr int ROW_UNKNOWN = INT_MIN;       // no verdict yet (calls with more rows than SMs clear row_out to this)

struct AcceptParams {
    const float *logits;
    const float *q;
    const int32_t *draft;
    const float *u_acc;
    const float *u_res;
    int B, K, rows, V, v_begin, n;
    float cfg_scale, temperature;
    int top_k;
    int vec_ok;
    int guided_in;     // logits is [B][rows][V] of guided logits instead of [2B][rows][V]
    int skip_mode;     // row_out was cleared: a row whose sequence is known to be rejected earlier does nothing
    int32_t *row_out;  // [B][rows]
    float *p_debug;
    int32_t *dev_status;
};

__device__ __forceinline__ float4 ld_stream4(const float *p)
{
    return __ldcs(reinterpret_cast<const float4 *>(p));
}

// Loads 4 consecutive floats starting at element e of a row of n valid elements; elements past
// the row end read as `fill`.
__device__ __forceinline__ float4 load4(const float *row, int e, int n, bool vec_ok, float fill)
{
    if (vec_ok && e + 3 < n) return ld_stream4(row + e);
    float4 r;
    r.x = e + 0 < n ? __ldcs(row + e + 0) : fill;
    r.y = e + 1 < n ? __ldcs(row + e + 1) : fill;
    r.z = e + 2 < n ? __ldcs(row + e + 2) : fill;
    r.w = e + 3 < n ? __ldcs(row + e + 3) : fill;
    return r;
}

// Guided logit in fp32: subtract, fused multiply-add, divide (three correctly rounded steps; a
// temperature of exactly 1 leaves the value as it is, so the divide is skipped).
// -inf in either stream gives -inf; NaN or +inf anywhere (inputs or result) gives -inf and a flag.
__device__ __forceinline__ float guided(float c, float u, float s, float T, bool unit_T, int &flags)
{
    if (fabsf(c) < CUDART_INF_F && fabsf(u) < CUDART_INF_F) {  // both finite: the common case
        float r = __fmaf_rn(s, __fsub_rn(c, u), u);
        if (!unit_T) r = __fdiv_rn(r, T);
        if (fabsf(r) < CUDART_INF_F) return r;
        if (r != -CUDART_INF_F) flags |= HAWK_DEV_NONFINITE;  // overflow to +inf or NaN
        return -CUDART_INF_F;
    }
    if ((c != c) || (u != u) || c == CUDART_INF_F || u == CUDART_INF_F) flags |= HAWK_DEV_NONFINITE;
    return -CUDART_INF_F;
}

// Order-preserving map between fp32 values (no NaN) and int32; it is its own inverse.
__device__ __forceinline__ int ordered_int(float v)
{
    const int k = __float_as_int(v);
    return k ^ ((k >> 31) & 0x7fffffff);
}
__device__ __forceinline__ float ordered_float(int k) { return __int_as_float(k ^ ((k >> 31) & 0x7fffffff)); }

// Scratch of the block-wide reductions.  Every call site has a slot of its own, so a reduction
// needs ONE barrier (publish, then read): with 32 warps a barrier costs some 400 cycles, and a
// second one per call only guarded the reuse of the scratch.
//   slot 0: range of the row          slot 1: range of a crowded bin (narrowing rounds)
//   slot 2: softmax sum               slot 3: residual mass of a rejected candidate (tree)
//   slot 4: bin search
// Two uses of the same slot are always separated by at least one other barrier.
constexpr int kRedSlots = 5;
template <int NT>
struct Scratch {
    float f[kRedSlots][32];
    int i[kRedSlots][3][32];
};

// Block-wide max, min and count: one redux instruction per value and level instead of shuffle trees.
template <int NT, int SLOT>
__device__ __forceinline__ void block_minmaxcount(float &mx, float &mn, int &cnt, Scratch<NT> &s)
{
    constexpr int kNW = NT / 32;
    int kmx = __reduce_max_sync(0xffffffffu, ordered_int(mx));
    int kmn = __reduce_min_sync(0xffffffffu, ordered_int(mn));
    cnt = __reduce_add_sync(0xffffffffu, cnt);
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    if (lane == 0) {
        s.i[SLOT][0][warp] = kmx;
        s.i[SLOT][1][warp] = kmn;
        s.i[SLOT][2][warp] = cnt;
    }
    __syncthreads();
    kmx = __reduce_max_sync(0xffffffffu, lane < kNW ? s.i[SLOT][0][lane] : ordered_int(-CUDART_INF_F));
    kmn = __reduce_min_sync(0xffffffffu, lane < kNW ? s.i[SLOT][1][lane] : ordered_int(CUDART_INF_F));
    cnt = __reduce_add_sync(0xffffffffu, lane < kNW ? s.i[SLOT][2][lane] : 0);
    mx = ordered_float(kmx);
    mn = ordered_float(kmn);
}

template <int NT, int SLOT>
__device__ __forceinline__ float block_sum(float v, Scratch<NT> &s)
{
    constexpr int kNW = NT / 32;
    v = hawk::warp_sum(v);
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    if (lane == 0) s.f[SLOT][warp] = v;
    __syncthreads();
    v = lane < kNW ? s.f[SLOT][lane] : 0.f;
    return hawk::warp_sum(v);
}

// Exclusive prefix sum of ints over the block in thread order; *total receives the block sum.  The
// warp totals go through shared memory once and every warp scans them for itself.
template <int NT, int SLOT>
__device__ __forceinline__ int block_exclusive_scan(int v, Scratch<NT> &s, int *total)
{
    constexpr int kNW = NT / 32;
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    int incl = v;
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) {
        const int up = __shfl_up_sync(0xffffffffu, incl, o);
        if (lane >= o) incl += up;
    }
    if (lane == 31) s.i[SLOT][0][warp] = incl;
    __syncthreads();
    const int w = lane < kNW ? s.i[SLOT][0][lane] : 0;
    int wi = w;
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) {
        const int up = __shfl_up_sync(0xffffffffu, wi, o);
        if (lane >= o) wi += up;
    }
    *total = __shfl_sync(0xffffffffu, wi, 31);
    return __shfl_sync(0xffffffffu, wi - w, warp) + (incl - v);
}

constexpr int kMaxChildren = 16;  // candidates verified at one tree node, at most

// Shared memory of one row block.
template <int NT, int VPT>
struct RowShared {
    int hist[kBins];
    float cand[kCandMax];
    Scratch<NT> red;
    float wt[VPT * (NT / 32)];
    float wbase[VPT * (NT / 32)];
    int bin, above, tok, ncand;
    float tau, pxe, total;
    int32_t *dbg_status;  // where the debug build's index checks report (set by the kernels; unused otherwise)
    int ctok[kMaxChildren];
    float cqx[kMaxChildren], cu[kMaxChildren];
};

// Reads the conditional and unconditional logit rows once and leaves the guided logits of the block's
// ids in registers (id of x[j][c]: 4 * (j * NT + tid) + c; ids past n hold -inf); also this thread's
// max, min and count of finite values.
// The common case runs without a branch: the guided value is computed for every id and replaced by
// -inf where an input or the result is not finite; which of those deserve the NONFINITE flag (NaN
// or +inf, as opposed to a plain -inf mask) is sorted out afterwards, and only by threads that met one.
// `full` (block-uniform): the row fills the block exactly and is 16-byte aligned, so no id needs a
// bounds check.
// GUIDED: lc already holds guided logits (the head projection combined the two
// streams); the caller passes temperature 1, so the arithmetic below returns every finite value as it
// is (fma(s, c - c, c) = c) and the row is read once.
template <int NT, int VPT, bool GUIDED>
__device__ __forceinline__ void row_load(const float *lc, const float *lu, int n, bool vec_ok, bool full,
                                         float cfg_scale, float temperature, float (&x)[VPT][4], float &mx,
                                         float &mn, int &cnt, int &flags)
{
    const int tid = threadIdx.x;
    const bool unit_T = temperature == 1.0f;
    mx = -CUDART_INF_F, mn = CUDART_INF_F, cnt = 0;
    float4 c4[VPT], u4[VPT];
    if (full) {
#pragma unroll
        for (int j = 0; j < VPT; ++j) {  // all loads in flight before the first use
            c4[j] = ld_stream4(lc + 4 * (j * NT + tid));
            u4[j] = GUIDED ? c4[j] : ld_stream4(lu + 4 * (j * NT + tid));
        }
    } else {
#pragma unroll
        for (int j = 0; j < VPT; ++j) {
            const int e0 = 4 * (j * NT + tid);
            c4[j] = e0 < n ? load4(lc, e0, n, vec_ok, -CUDART_INF_F) : make_float4(-CUDART_INF_F, -CUDART_INF_F, -CUDART_INF_F, -CUDART_INF_F);
            u4[j] = (!GUIDED && e0 < n) ? load4(lu, e0, n, vec_ok, -CUDART_INF_F) : c4[j];
        }
    }
    bool odd = false;  // met an id whose inputs or result are not finite
#pragma unroll
    for (int j = 0; j < VPT; ++j) {
        const float cs[4] = {c4[j].x, c4[j].y, c4[j].z, c4[j].w}, us[4] = {u4[j].x, u4[j].y, u4[j].z, u4[j].w};
#pragma unroll
        for (int c = 0; c < 4; ++c) {
            float r = __fmaf_rn(cfg_scale, __fsub_rn(cs[c], us[c]), us[c]);
            if (!unit_T) r = __fdiv_rn(r, temperature);
            const bool ok = (fabsf(cs[c]) < CUDART_INF_F) & (fabsf(us[c]) < CUDART_INF_F) & (fabsf(r) < CUDART_INF_F);
            odd |= !ok;
            r = ok ? r : -CUDART_INF_F;
            x[j][c] = r;
            mx = fmaxf(mx, r);                          // -inf leaves the maximum alone
            mn = fminf(mn, ok ? r : CUDART_INF_F);
            cnt += ok;
        }
    }
    if (odd) {  // rare: read those ids again and look exactly (ids past the row end read as -inf: no flag)
#pragma unroll 1
        for (int j = 0; j < VPT; ++j) {
            const int e0 = 4 * (j * NT + tid);
            if (e0 >= n) break;
            const float4 a = load4(lc, e0, n, vec_ok, -CUDART_INF_F), b = GUIDED ? a : load4(lu, e0, n, vec_ok, -CUDART_INF_F);
            int fl = 0;
            (void)guided(a.x, b.x, cfg_scale, temperature, unit_T, fl);
            (void)guided(a.y, b.y, cfg_scale, temperature, unit_T, fl);
            (void)guided(a.z, b.z, cfg_scale, temperature, unit_T, fl);
            (void)guided(a.w, b.w, cfg_scale, temperature, unit_T, fl);
            flags |= fl;
        }
    }
}

// Top-k threshold of a row held in registers: the top_k-th largest finite value (exact; ties at it
// are all kept).  -inf when nothing is to be filtered.  mn, mx, cnt: block-wide range and count.
template <int NT, int VPT>
__device__ __forceinline__ float row_topk(const float (&x)[VPT][4], float mn, float mx, int cnt, int top_k,
                                          RowShared<NT, VPT> &sh)
{
    constexpr int BPT = kBins / NT;  // histogram bins per thread
    static_assert(kBins % NT == 0 && BPT >= 1, "bins must split evenly over the block");
    constexpr int NW = NT / 32;
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    (void)lane; (void)warp; (void)NW;
    float tau = -CUDART_INF_F;
    if (top_k > 0 && top_k < cnt) {
        float lo = mn, hi = mx;
        int k = top_k;
        for (int round = 0; round < kMaxRounds; ++round) {
            if (!(hi > lo)) {
                tau = hi;
                break;
            }
            // histogram of the values in [lo, hi]: bin 0 holds the largest
            const float scale = static_cast<float>(kBins) / (hi - lo);
#pragma unroll
            for (int t = 0; t < BPT; ++t) sh.hist[t * NT + tid] = 0;
            if (tid == 0) sh.ncand = 0;
            __syncthreads();
            int bins[VPT][4];  // bin of every value held (-1: outside [lo, hi])
#pragma unroll
            for (int j = 0; j < VPT; ++j)
#pragma unroll
                for (int c = 0; c < 4; ++c) {
                    const float v = x[j][c];
                    const bool in = v >= lo && v <= hi;
                    bins[j][c] = in ? min(kBins - 1, static_cast<int>((hi - v) * scale)) : -1;
                    if (in && HAWK_IN_BOUNDS(sh.dbg_status, bins[j][c], kBins)) atomicAdd(&sh.hist[bins[j][c]], 1);
                }
            __syncthreads();
            int local = 0;
#pragma unroll
            for (int t = 0; t < BPT; ++t) local += sh.hist[tid * BPT + t];
            int total;
            const int excl = block_exclusive_scan<NT, 4>(local, sh.red, &total);
            if (excl < k && k <= excl + local) {  // exactly one thread: one of its bins holds the k-th largest
                int run = excl;
#pragma unroll
                for (int t = 0; t < BPT; ++t) {
                    const int h = sh.hist[tid * BPT + t];
                    if (run < k && k <= run + h) {
                        sh.bin = tid * BPT + t;
                        sh.above = run;
                    }
                    run += h;
                }
            }
            __syncthreads();
            const int bstar = sh.bin, kk = k - sh.above, C = sh.hist[bstar];
            if (C <= kCandMax) {
                // rank the members of the bin exactly: the kk-th largest of them is the threshold.
                // They are few (a 1024th of the value range), so gathering them through one shared
                // counter is cheaper than a block-wide prefix sum (measured).
#pragma unroll
                for (int j = 0; j < VPT; ++j)
#pragma unroll
                    for (int c = 0; c < 4; ++c)
                        if (bins[j][c] == bstar) {
                            const int at = atomicAdd(&sh.ncand, 1);
                            if (HAWK_IN_BOUNDS(sh.dbg_status, at, kCandMax)) sh.cand[at] = x[j][c];
                        }
                __syncthreads();
                if (C <= 32) {  // the usual case: one warp ranks them, all 32 exchanges in flight at once
                    if (warp == 0) {
                        const float v = lane < C ? sh.cand[lane] : -CUDART_INF_F;
                        int gt = 0, ge = 0;
#pragma unroll 8
                        for (int m = 0; m < 32; ++m) {
                            const float w = __shfl_sync(0xffffffffu, v, m);  // lanes >= C hold -inf: never > or >= a member
                            gt += w > v;
                            ge += (w >= v) & (m < C);
                        }
                        if (lane < C && gt < kk && kk <= ge) sh.tau = v;
                    }
                } else {
                    for (int t = tid; t < C; t += NT) {
                        const float v = sh.cand[t];
                        int gt = 0, ge = 0;
                        for (int m = 0; m < C; ++m) {
                            const float w = sh.cand[m];
                            gt += w > v;
                            ge += w >= v;
                        }
                        if (gt < kk && kk <= ge) sh.tau = v;  // several threads may hold the same value
                    }
                }
                __syncthreads();
                tau = sh.tau;
                break;
            }
            // too many members share the bin: narrow the range to their values and repeat
            float nmx = -CUDART_INF_F, nmn = CUDART_INF_F;
            int dummy = 0;
#pragma unroll
            for (int j = 0; j < VPT; ++j)
#pragma unroll
                for (int c = 0; c < 4; ++c)
                    if (bins[j][c] == bstar) {
                        nmx = fmaxf(nmx, x[j][c]);
                        nmn = fminf(nmn, x[j][c]);
                    }
            block_minmaxcount<NT, 1>(nmx, nmn, dummy, sh.red);
            lo = nmn;
            hi = nmx;
            k = kk;
            if (round == kMaxRounds - 1) tau = hi;  // unreachable for fp32 ranges; keeps tau defined
        }
    }

    return tau;
}

// x becomes exp(l - max) for the ids kept by the threshold (0 for the others); returns the block-wide sum.
template <int NT, int VPT>
__device__ __forceinline__ float row_softmax(float (&x)[VPT][4], float tau, float mx, RowShared<NT, VPT> &sh)
{
    constexpr float kLog2e = 1.4426950408889634f;
    float zsum = 0.f;
#pragma unroll
    for (int j = 0; j < VPT; ++j)
#pragma unroll
        for (int c = 0; c < 4; ++c) {
            const float v = x[j][c];  // -inf gives exp2(-inf) = 0
            const float e = v >= tau ? hawk::fast_exp2((v - mx) * kLog2e) : 0.f;
            x[j][c] = e;
            zsum += e;
        }
    return block_sum<NT, 2>(zsum, sh.red);
}

// Running sums of the non-negative weights rr in ascending id order: sj = sum of each group of 4,
// incl = inclusive scan of sj over the warp, sh.wbase = mass before each (group row, warp); returns the
// total mass.  Also resets sh.tok for row_search().
template <int NT, int VPT>
__device__ __forceinline__ float row_mass(const float (&rr)[VPT][4], float (&sj)[VPT], float (&incl)[VPT],
                                          RowShared<NT, VPT> &sh)
{
    static_assert(VPT * (NT / 32) <= NT, "warp totals of the scan must fit one block-wide scan");
    constexpr int NW = NT / 32;
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    (void)lane; (void)warp; (void)NW;
#pragma unroll
    for (int j = 0; j < VPT; ++j) sj[j] = ((rr[j][0] + rr[j][1]) + rr[j][2]) + rr[j][3];
#pragma unroll
    for (int j = 0; j < VPT; ++j) {
        float v = sj[j];
#pragma unroll
        for (int o = 1; o < 32; o <<= 1) {
            const float up = __shfl_up_sync(0xffffffffu, v, o);
            if (lane >= o) v += up;
        }
        incl[j] = v;
        if (lane == 31) sh.wt[j * NW + warp] = v;
    }
    __syncthreads();
    if (warp == 0) {  // exclusive prefix of the VPT * NW warp totals (ascending id order), by one warp
        constexpr int E = VPT * NW, PER = (E + 31) / 32;
        float ent[PER], run = 0.f;
#pragma unroll
        for (int t = 0; t < PER; ++t) {
            ent[t] = lane * PER + t < E ? sh.wt[lane * PER + t] : 0.f;
            run += ent[t];
        }
        float incl_l = run;
#pragma unroll
        for (int o = 1; o < 32; o <<= 1) {
            const float up = __shfl_up_sync(0xffffffffu, incl_l, o);
            if (lane >= o) incl_l += up;
        }
        float base = incl_l - run;
#pragma unroll
        for (int t = 0; t < PER; ++t) {
            if (lane * PER + t < E) sh.wbase[lane * PER + t] = base;
            base += ent[t];
        }
        if (lane == 31) sh.total = incl_l;
        if (lane == 0) sh.tok = 0x7fffffff;
    }
    __syncthreads();
    return sh.total;
}

// Inverse CDF: the smallest id (local to the valid range) whose running sum of rr exceeds tl; if
// rounding leaves none, the last id with mass; -1 if no id has mass.
template <int NT, int VPT>
__device__ __forceinline__ int row_search(const float (&rr)[VPT][4], const float (&sj)[VPT],
                                          const float (&incl)[VPT], float tl, RowShared<NT, VPT> &sh)
{
    constexpr int NW = NT / 32;
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    (void)lane; (void)warp; (void)NW;
    // pass 0: elements where the running sum crosses tl; pass 1 (only if the block-wide sums
    // disagree at a thread boundary): the first element whose running sum exceeds tl
    for (int pass = 0; pass < 2; ++pass) {
#pragma unroll
        for (int j = 0; j < VPT; ++j) {
            const float excl = sh.wbase[j * NW + warp] + (incl[j] - sj[j]);
            const bool look = pass == 0 ? (excl <= tl && excl + sj[j] > tl) : (excl + sj[j] > tl);
            if (look) {
                const int e0 = 4 * (j * NT + tid);
                const float r0 = rr[j][0], r1 = rr[j][1], r2 = rr[j][2], r3 = rr[j][3];
                const float c0 = excl + r0, c1 = excl + (r0 + r1), c2 = excl + ((r0 + r1) + r2);
                const float c3 = excl + (((r0 + r1) + r2) + r3);
                int hit = -1;  // an id without mass is never drawn
                if (r0 > 0.f && c0 > tl) hit = 0;
                else if (r1 > 0.f && c1 > tl) hit = 1;
                else if (r2 > 0.f && c2 > tl) hit = 2;
                else if (r3 > 0.f && c3 > tl) hit = 3;
                if (hit >= 0) atomicMin(&sh.tok, e0 + hit);
            }
        }
        __syncthreads();
        if (sh.tok != 0x7fffffff) break;
        __syncthreads();
    }
    int tok = sh.tok;
    if (tok == 0x7fffffff) {  // rounding left no running sum above tl: the last id with mass
        __syncthreads();
        if (tid == 0) sh.tok = -1;
        __syncthreads();
#pragma unroll
        for (int j = 0; j < VPT; ++j) {
            const int e0 = 4 * (j * NT + tid);
            if (sj[j] > 0.f) {
                int last = -1;
#pragma unroll
                for (int c = 0; c < 4; ++c)
                    if (rr[j][c] > 0.f) last = e0 + c;
                if (last >= 0) atomicMax(&sh.tok, last);
            }
        }
        __syncthreads();
        tok = sh.tok;
    }
    return tok;
}

// Chain verification: one block per (sequence, draft position) row.
// NT threads, VPT float4 loads per thread: the block holds up to 4 * NT * VPT valid ids of its row.
template <int NT, int VPT, bool GUIDED>
__global__ void __launch_bounds__(NT) accept_rows_kernel(const AcceptParams P)
{
    __shared__ RowShared<NT, VPT> sh;
    const int tid = threadIdx.x;
    if (tid == 0) sh.dbg_status = P.dev_status;  // (published by the first block-wide barrier, long before its first use)
    hawk::allow_dependent_launch();
    hawk::grid_dependency_wait();

    const int row = blockIdx.x;  // position-major: all rows of position 0 first
    const int i = row / P.B, b = row - i * P.B;
    // A chain ends at its first rejection, so the rows behind it are never looked at.  With more rows than SMs
    // the blocks of the later positions start after those of the earlier ones have finished: such a block looks
    // at the verdicts its sequence already has and, if one of them is a rejection, has nothing to do.  A verdict
    // that is not visible yet only costs the skipped work; the result does not depend on what is seen here.
    if (P.skip_mode && i > 0) {
        int rejected = 0;
        if (tid < i) {
            const int c = *reinterpret_cast<const volatile int32_t *>(&P.row_out[b * P.rows + tid]);
            rejected = (c != ROW_UNKNOWN && c != ROW_ACCEPTED) ? 1 : 0;
        }
        if (__syncthreads_or(rejected)) return;
    }
    const bool bonus = (i == P.K);
    const int n = P.n;
    const bool vec_ok = P.vec_ok != 0;
    const float *lc = P.logits + (static_cast<size_t>(b) * P.rows + i) * P.V + P.v_begin;
    const float *lu = GUIDED ? nullptr : P.logits + (static_cast<size_t>(P.B + b) * P.rows + i) * P.V + P.v_begin;
    const float *qrow = bonus ? nullptr : P.q + (static_cast<size_t>(b) * P.K + i) * P.V + P.v_begin;
    int flags = 0;

    // draft id and uniforms: requested before the rows, so that they have arrived when the rows have
    int xd = bonus ? P.v_begin : P.draft[b * P.K + i];
    const float u_acc = bonus ? 0.f : P.u_acc[b * P.K + i];
    const float u_res = P.u_res[b * (P.K + 1) + i];

    float x[VPT][4];
    float mx, mn;
    int cnt;
    row_load<NT, VPT, GUIDED>(lc, lu, n, vec_ok, vec_ok && n == 4 * NT * VPT, P.cfg_scale, P.temperature, x, mx, mn, cnt, flags);

    float qx = 0.f;
    if (!bonus) {
        if (xd < P.v_begin || xd >= P.v_begin + n) {
            flags |= HAWK_DEV_BAD_DRAFT;
            xd = xd < P.v_begin ? P.v_begin : P.v_begin + n - 1;
        }
        xd -= P.v_begin;
        if (HAWK_IN_BOUNDS(P.dev_status, xd, n)) qx = qrow[xd];
    }
    if (flags && P.dev_status) atomicOr(P.dev_status, flags);

    block_minmaxcount<NT, 0>(mx, mn, cnt, sh.red);

    if (cnt == 0) {  // nothing has mass: p == 0 everywhere, the draft is rejected, no token exists
        if (P.p_debug) {
            float *pd = P.p_debug + (static_cast<size_t>(b) * P.rows + i) * P.V + P.v_begin;
            for (int e = tid; e < n; e += NT) pd[e] = 0.f;
        }
        if (tid == 0 && HAWK_IN_BOUNDS(P.dev_status, b * P.rows + i, P.B * P.rows)) P.row_out[b * P.rows + i] = ROW_REJECTED_NO_TOKEN;
        return;
    }

    const float tau = row_topk<NT, VPT>(x, mn, mx, cnt, P.top_k, sh);

    // ---- softmax over what is kept: x becomes exp(l - max), unnormalised
    if (!bonus && tid == ((xd >> 2) % NT)) {  // the thread that holds the draft id publishes exp(l_x - max)
#pragma unroll
        for (int j = 0; j < VPT; ++j)
#pragma unroll
            for (int c = 0; c < 4; ++c)
                if (4 * (j * NT + tid) + c == xd)
                    sh.pxe = x[j][c] >= tau ? hawk::fast_exp2((x[j][c] - mx) * 1.4426950408889634f) : 0.f;
    }
    const float Z = row_softmax<NT, VPT>(x, tau, mx, sh);  // its barriers publish sh.pxe
    const float pxe = sh.pxe;
    const float invZ = 1.0f / Z;

    if (P.p_debug) {
        float *pd = P.p_debug + (static_cast<size_t>(b) * P.rows + i) * P.V + P.v_begin;
#pragma unroll
        for (int j = 0; j < VPT; ++j)
#pragma unroll
            for (int c = 0; c < 4; ++c) {
                const int e = 4 * (j * NT + tid) + c;
                if (e < n && HAWK_IN_BOUNDS(P.dev_status, (static_cast<long long>(b) * P.rows + i) * P.V + P.v_begin + e,
                                            static_cast<long long>(P.B) * P.rows * P.V))
                    pd[e] = x[j][c] * invZ;
            }
    }

    // ---- acceptance test on the draft token
    if (!bonus) {
        const float px = pxe * invZ;
        const bool accepted = static_cast<double>(u_acc) * static_cast<double>(qx) < static_cast<double>(px);
        if (accepted) {
            if (tid == 0 && HAWK_IN_BOUNDS(P.dev_status, b * P.rows + i, P.B * P.rows)) P.row_out[b * P.rows + i] = ROW_ACCEPTED;
            return;
        }
    }

    // ---- rejected (or bonus row): inverse-CDF draw from max(0, p - q), or from p itself
    // The rejection itself is published at once (the token follows): rows of later positions that start while this
    // block is still drawing its token see that their chain has ended and do nothing.
    if (P.skip_mode && !bonus && tid == 0)
        *reinterpret_cast<volatile int32_t *>(&P.row_out[b * P.rows + i]) = ROW_REJECTED_NO_TOKEN;
    bool use_q = !bonus;
    for (int attempt = 0; attempt < 2; ++attempt) {
        float rr[VPT][4], sj[VPT], incl[VPT];  // residual weights of this thread's ids and their running sums
        {
            float4 q4[VPT];
#pragma unroll
            for (int j = 0; j < VPT; ++j) {  // all loads in flight before the first use
                const int e0 = 4 * (j * NT + tid);
                q4[j] = (use_q && e0 < n) ? load4(qrow, e0, n, vec_ok, 0.f) : make_float4(0.f, 0.f, 0.f, 0.f);
            }
#pragma unroll
            for (int j = 0; j < VPT; ++j) {
                rr[j][0] = fmaxf(0.f, x[j][0] * invZ - q4[j].x);
                rr[j][1] = fmaxf(0.f, x[j][1] * invZ - q4[j].y);
                rr[j][2] = fmaxf(0.f, x[j][2] * invZ - q4[j].z);
                rr[j][3] = fmaxf(0.f, x[j][3] * invZ - q4[j].w);
            }
        }
        const float total = row_mass<NT, VPT>(rr, sj, incl, sh);
        if (use_q && !(total > 0.f)) {  // p <= q everywhere: draw from p with the same uniform
            use_q = false;
            continue;
        }
        const int tok = row_search<NT, VPT>(rr, sj, incl, u_res * total, sh);
        if (tid == 0 && HAWK_IN_BOUNDS(P.dev_status, b * P.rows + i, P.B * P.rows) &&
            (tok == -1 || HAWK_IN_BOUNDS(P.dev_status, tok, n)))
            P.row_out[b * P.rows + i] = tok >= 0 ? P.v_begin + tok : ROW_REJECTED_NO_TOKEN;
        return;
    }
}

// ------------------------------------------------------------------------------------------------
// Tree verification (several candidates per depth, each with its own draft distribution; Sec. 4.2,
// Eq. "recur"): one block per (sequence, tree node).  The block computes the node's target
// distribution exactly as above and then verifies the node's children in order, keeping the
// refined target max(0, p - q) un-normalised in registers with its mass as a scalar.  Its verdict is
// the child that passed, or the correction token drawn from the target as refined by every rejection.
// Every node is judged, whether or not the walk will reach it; a second kernel follows the verdicts
// from the root.
struct TreeParams {
    const float *logits;        // [2B][N][V]
    const float *q;             // [B][NQ][V]
    const int32_t *node_token;  // [B][N]
    const int32_t *node_q;      // [N]
    const int32_t *child_begin; // [N + 1]
    const float *u_acc;         // [B][N]
    const float *u_res;         // [B][N]
    int B, N, NQ, V, v_begin, n;
    float cfg_scale, temperature;
    int top_k;
    int vec_ok;
    int guided_in;     // logits is [B][N][V] of guided logits instead of [2B][N][V]
    int skip_mode;     // verdicts were cleared and `parent` filled in: a node its parent did not pick does nothing
    const int32_t *parent;  // [N], written by tree_prepare_kernel
    int32_t *verdict;  // [B][N]: >= 0 the child that passed; -1 stop without a token; <= -2 stop, token = -v - 2
    int32_t *dev_status;
};

template <int NT, int VPT, bool GUIDED>
__global__ void __launch_bounds__(NT) tree_rows_kernel(const TreeParams P)
{
    __shared__ RowShared<NT, VPT> sh;
    __shared__ int s_cq[kMaxChildren];
    const int tid = threadIdx.x;
    if (tid == 0) sh.dbg_status = P.dev_status;
    hawk::allow_dependent_launch();
    hawk::grid_dependency_wait();

    const int row = blockIdx.x;  // node-major
    const int node = row / P.B, b = row - node * P.B;
    // The walk reaches a node only as the child its parent picked.  With more rows than SMs the blocks of the
    // deeper nodes start after their parents have finished: a node whose parent is known to have picked
    // another child, to have stopped, or to be unreachable itself, is marked unreachable and does nothing.
    if (P.skip_mode && node > 0) {
        int dead = 0;
        if (tid == 0) {
            const int par = P.parent[node];
            if (par >= 0 && par < node) {
                const int v = *reinterpret_cast<const volatile int32_t *>(&P.verdict[b * P.N + par]);
                dead = (v != ROW_UNKNOWN && v != node) ? 1 : 0;
            }
        }
        if (__syncthreads_or(dead)) {
            if (tid == 0) P.verdict[b * P.N + node] = -1;
            return;
        }
    }
    const int n = P.n;
    const bool vec_ok = P.vec_ok != 0;
    const float *lc = P.logits + (static_cast<size_t>(b) * P.N + node) * P.V + P.v_begin;
    const float *lu = GUIDED ? nullptr : P.logits + (static_cast<size_t>(P.B + b) * P.N + node) * P.V + P.v_begin;
    int flags = 0;

    // children of the node; ids must grow along the walk so that it ends
    int cb = P.child_begin[node], ce = P.child_begin[node + 1];
    if (cb < ce) {
        const int cb1 = max(node + 1, min(cb, P.N));
        const int ce1 = max(cb1, min(ce, min(P.N, cb1 + kMaxChildren)));
        if (cb1 != cb || ce1 != ce) flags |= HAWK_DEV_BAD_TREE;  // clamped: the walk still ends
        cb = cb1;
        ce = ce1;
    } else {  // a leaf (begin == end, whatever the value)
        if (cb > ce) flags |= HAWK_DEV_BAD_TREE;
        ce = cb;
    }
    const int nc = ce - cb;
    // this thread's child (threads 0 .. nc-1): token, draft row and uniform, requested before the rows
    int my_tok = 0, my_q = 0;
    float my_u = 0.f, my_qx = 0.f;
    if (tid < nc) {
        my_tok = P.node_token[b * P.N + cb + tid];
        my_q = P.node_q[cb + tid];
        my_u = P.u_acc[b * P.N + cb + tid];
    }
    const float u_res = P.u_res[b * P.N + node];

    float x[VPT][4];
    float mx, mn;
    int cnt;
    row_load<NT, VPT, GUIDED>(lc, lu, n, vec_ok, vec_ok && n == 4 * NT * VPT, P.cfg_scale, P.temperature, x, mx, mn, cnt, flags);

    if (tid < nc) {
        if (my_tok < P.v_begin || my_tok >= P.v_begin + n) {
            flags |= HAWK_DEV_BAD_DRAFT;
            my_tok = my_tok < P.v_begin ? P.v_begin : P.v_begin + n - 1;
        }
        my_tok -= P.v_begin;
        if (my_q < 0 || my_q >= P.NQ) {
            flags |= HAWK_DEV_BAD_TREE;
            my_q = max(0, min(my_q, P.NQ - 1));
        }
        if (HAWK_IN_BOUNDS(P.dev_status, my_tok, n) && HAWK_IN_BOUNDS(P.dev_status, my_q, P.NQ))
            my_qx = P.q[(static_cast<size_t>(b) * P.NQ + my_q) * P.V + P.v_begin + my_tok];
    }
    if (flags && P.dev_status) atomicOr(P.dev_status, flags);

    block_minmaxcount<NT, 0>(mx, mn, cnt, sh.red);
    if (cnt == 0) {  // nothing has mass: every candidate is rejected and no token exists
        if (tid == 0) P.verdict[b * P.N + node] = -1;
        return;
    }
    const float tau = row_topk<NT, VPT>(x, mn, mx, cnt, P.top_k, sh);
    float mass = row_softmax<NT, VPT>(x, tau, mx, sh);  // x: un-normalised target, p = x / mass
    if (tid < nc) {  // the children's scalars have long arrived
        sh.ctok[tid] = my_tok;
        sh.cqx[tid] = my_qx;
        sh.cu[tid] = my_u;
        s_cq[tid] = my_q;
    }
    __syncthreads();

    for (int ci = 0; ci < nc; ++ci) {
        const int xd = sh.ctok[ci];
        if (tid == ((xd >> 2) % NT)) {  // the thread that holds the candidate's id
#pragma unroll
            for (int j = 0; j < VPT; ++j)
#pragma unroll
                for (int c = 0; c < 4; ++c)
                    if (4 * (j * NT + tid) + c == xd) sh.pxe = x[j][c];
        }
        __syncthreads();
        const float px = sh.pxe / mass;
        const bool accepted = static_cast<double>(sh.cu[ci]) * static_cast<double>(sh.cqx[ci]) < static_cast<double>(px);
        if (accepted) {
            if (tid == 0 && HAWK_IN_BOUNDS(P.dev_status, b * P.N + node, P.B * P.N) && HAWK_IN_BOUNDS(P.dev_status, cb + ci, P.N))
                P.verdict[b * P.N + node] = cb + ci;
            return;
        }
        // rejected: target <- max(0, p - q), kept un-normalised as max(0, x - mass * q)
        const float *qrow = P.q + (static_cast<size_t>(b) * P.NQ + s_cq[ci]) * P.V + P.v_begin;
        float rr[VPT][4], rsum = 0.f;
        {
            float4 q4[VPT];
#pragma unroll
            for (int j = 0; j < VPT; ++j) {
                const int e0 = 4 * (j * NT + tid);
                q4[j] = e0 < n ? load4(qrow, e0, n, vec_ok, 0.f) : make_float4(0.f, 0.f, 0.f, 0.f);
            }
#pragma unroll
            for (int j = 0; j < VPT; ++j) {
                rr[j][0] = fmaxf(0.f, fmaf(-mass, q4[j].x, x[j][0]));
                rr[j][1] = fmaxf(0.f, fmaf(-mass, q4[j].y, x[j][1]));
                rr[j][2] = fmaxf(0.f, fmaf(-mass, q4[j].z, x[j][2]));
                rr[j][3] = fmaxf(0.f, fmaf(-mass, q4[j].w, x[j][3]));
                rsum += (rr[j][0] + rr[j][1]) + (rr[j][2] + rr[j][3]);
            }
        }
        rsum = block_sum<NT, 3>(rsum, sh.red);
        if (rsum > 0.f) {  // a residual without mass (p <= q everywhere) leaves the target as it is
            mass = rsum;
#pragma unroll
            for (int j = 0; j < VPT; ++j)
#pragma unroll
                for (int c = 0; c < 4; ++c) x[j][c] = rr[j][c];
        }
    }

    // ---- every candidate rejected (or a leaf): draw the correction token from the target as refined
    // (the outcome "no child was picked" is published at once, the token follows: the children's blocks that start
    // in the meantime see that the walk cannot reach them)
    if (P.skip_mode && nc > 0 && tid == 0) *reinterpret_cast<volatile int32_t *>(&P.verdict[b * P.N + node]) = -1;
    float sj[VPT], incl[VPT];
    const float total = row_mass<NT, VPT>(x, sj, incl, sh);
    int tok = -1;
    if (total > 0.f) tok = row_search<NT, VPT>(x, sj, incl, u_res * total, sh);
    if (tid == 0 && HAWK_IN_BOUNDS(P.dev_status, b * P.N + node, P.B * P.N)) P.verdict[b * P.N + node] = tok >= 0 ? -(P.v_begin + tok) - 2 : -1;
}

// ------------------------------------------------------------------------------------------------
// Drawing the candidates (Sec. 4.2: the candidates of the tree are samples from the distributions of
// the spatial sampling pool): one block per (sequence, pool row) draws one token by inverse CDF in
// ascending id, with the same scan and search as the correction token above.
template <int NT, int VPT>
__global__ void __launch_bounds__(NT) pool_sample_kernel(const float *pool_q, const float *u, const int32_t *node_q,
                                                         int32_t *node_token, int NQ, int N, int V, int v_begin, int n,
                                                         int vec_ok, int32_t *dev_status)
{
    __shared__ RowShared<NT, VPT> sh;
    const int tid = threadIdx.x;
    if (tid == 0) sh.dbg_status = dev_status;
    hawk::allow_dependent_launch();
    hawk::grid_dependency_wait();
    const float *qrow = pool_q + static_cast<size_t>(blockIdx.x) * V + v_begin;
    const float ur = u[blockIdx.x];
    float x[VPT][4], sj[VPT], incl[VPT];
#pragma unroll
    for (int j = 0; j < VPT; ++j) {
        const int e0 = 4 * (j * NT + tid);
        const float4 q4 = e0 < n ? load4(qrow, e0, n, vec_ok != 0, 0.f) : make_float4(0.f, 0.f, 0.f, 0.f);
        x[j][0] = fmaxf(q4.x, 0.f);  // (a NaN weight counts as none)
        x[j][1] = fmaxf(q4.y, 0.f);
        x[j][2] = fmaxf(q4.z, 0.f);
        x[j][3] = fmaxf(q4.w, 0.f);
    }
    const float total = row_mass<NT, VPT>(x, sj, incl, sh);
    int tok = -1;
    if (total > 0.f) tok = row_search<NT, VPT>(x, sj, incl, ur * total, sh);
    // every tree node that stands for this pool row carries the draw (the root, node 0, carries 0); a node_q
    // entry outside [0, NQ) is served by the first or the last row and flagged
    const int b = blockIdx.x / NQ, r = blockIdx.x - b * NQ;
    const int token = tok >= 0 ? v_begin + tok : -1;
    int bad = 0;
    for (int node = tid; node < N; node += NT) {
        if (node == 0) {
            if (r == 0) node_token[b * N] = 0;
            continue;
        }
        const int want = node_q[node];
        bad |= (want < 0 || want >= NQ) ? 1 : 0;
        if (max(0, min(want, NQ - 1)) == r && (token == -1 || HAWK_IN_BOUNDS(dev_status, token - v_begin, n)))
            node_token[b * N + node] = token;
    }
    if (bad && dev_status) atomicOr(dev_status, HAWK_DEV_BAD_TREE);
}

// For calls with more rows than SMs: marks every verdict "unknown" and writes each node's parent (the
// child ranges clamped exactly as tree_rows_kernel clamps them).
__global__ void tree_prepare_kernel(int32_t *verdict, int32_t *parent, const int32_t *child_begin, int B, int N)
{
    hawk::allow_dependent_launch();
    hawk::grid_dependency_wait();
    const int idx = blockIdx.x * blockDim.x + threadIdx.x;
    if (idx < B * N) verdict[idx] = ROW_UNKNOWN;
    if (idx == 0) parent[0] = -1;
    if (idx < N) {
        int cb = child_begin[idx], ce = child_begin[idx + 1];
        if (cb < ce) {
            cb = max(idx + 1, min(cb, N));
            ce = max(cb, min(ce, min(N, cb + kMaxChildren)));
            for (int c = cb; c < ce; ++c) parent[c] = idx;
        }
    }
}

// One thread per sequence: follows the verdicts from the root.
__global__ void tree_walk_kernel(const int32_t *verdict, int B, int N, int max_depth, int32_t *accept_len,
                                 int32_t *out_token, int32_t *path, int32_t *dev_status)
{
    hawk::allow_dependent_launch();
    hawk::grid_dependency_wait();
    const int b = blockIdx.x * blockDim.x + threadIdx.x;
    if (b >= B) return;
    int node = 0, depth = 0, tok = -1;
    for (int step = 0; step < N; ++step) {
        const int v = verdict[b * N + node];
        if (v < 0) {
            tok = v <= -2 ? -v - 2 : -1;
            break;
        }
        if (v <= node || v >= N) {  // cannot happen with verdicts of tree_rows_kernel; never loop
            if (dev_status) atomicOr(dev_status, HAWK_DEV_BAD_TREE);
            break;
        }
        if (path && depth < max_depth && HAWK_IN_BOUNDS(dev_status, b * max_depth + depth, B * max_depth)) path[b * max_depth + depth] = v;
        ++depth;
        node = v;
    }
    if (path)
        for (int d = depth; d < max_depth; ++d) path[b * max_depth + d] = -1;
    accept_len[b] = depth;
    out_token[b] = tok;
}

// One thread per sequence: the first rejected row decides accept_len and the correction token.
// Marks every row "no verdict yet" (after the dependency wait: the workspace may be memory that the preceding
// kernel in the stream still uses).
__global__ void accept_clear_kernel(int32_t *row_out, int n)
{
    hawk::allow_dependent_launch();
    hawk::grid_dependency_wait();
    const int idx = blockIdx.x * blockDim.x + threadIdx.x;
    if (idx < n) row_out[idx] = ROW_UNKNOWN;
}

__global__ void accept_finalize_kernel(const int32_t *row_out, int B, int K, int rows, int32_t *accept_len,
                                       int32_t *out_token)
{
    hawk::allow_dependent_launch();
    hawk::grid_dependency_wait();
    const int b = blockIdx.x * blockDim.x + threadIdx.x;
    if (b >= B) return;
    int len = K, tok = -1;
    for (int i = 0; i < K; ++i) {
        const int r = row_out[b * rows + i];
        if (r != ROW_ACCEPTED) {
            len = i;
            tok = r >= 0 ? r : -1;
            break;
        }
    }
    if (len == K && rows > K) {
        const int r = row_out[b * rows + K];
        tok = r >= 0 ? r : -1;
    }
    accept_len[b] = len;
    out_token[b] = tok;
}


template <int NT, int VPT>
cudaError_t launch_rows(const AcceptParams &P, int grid, cudaStream_t stream)
{
    if (P.guided_in)
        return hawk_host::launch_dependent(accept_rows_kernel<NT, VPT, true>, dim3(grid), dim3(NT), 0, stream, P);
    return hawk_host::launch_dependent(accept_rows_kernel<NT, VPT, false>, dim3(grid), dim3(NT), 0, stream, P);
}

template <int NT, int VPT>
cudaError_t launch_tree_rows(const TreeParams &P, int grid, cudaStream_t stream)
{
    if (P.guided_in)
        return hawk_host::launch_dependent(tree_rows_kernel<NT, VPT, true>, dim3(grid), dim3(NT), 0, stream, P);
    return hawk_host::launch_dependent(tree_rows_kernel<NT, VPT, false>, dim3(grid), dim3(NT), 0, stream, P);
}

}  // namespace

extern "C" size_t hawk_cfg_accept_workspace_bytes(int B, int K, int V)
{
    (void)V;
    if (B <= 0 || K <= 0) return 0;
    return static_cast<size_t>(B) * static_cast<size_t>(K + 1) * sizeof(int32_t);
}

hawk_status hawk_host::check_cfg_accept_args(const float *logits, const float *q_probs, const int32_t *draft,
                                             const float *u_accept, const float *u_resample, int B, int K, int V,
                                             int v_begin, int v_end, float cfg_scale, float temperature,
                                             const int32_t *accept_len, const int32_t *out_token, const float *p_debug,
                                             const void *workspace, size_t workspace_bytes)
{
    if (B < 0 || K < 0 || V < 0) return HAWK_ERR_SHAPE;
    if (B == 0) return HAWK_OK;
    if (!logits || !q_probs || !draft || !u_accept || !u_resample || !accept_len || !out_token) return HAWK_ERR_NULL;
    if (v_begin < 0 || v_end > V || v_begin >= v_end) return HAWK_ERR_SHAPE;
    if (K < 1 || K > 16) return HAWK_ERR_UNSUPPORTED;
    const int n = v_end - v_begin;
    if (n > 32768) return HAWK_ERR_UNSUPPORTED;  // one row must fit one block's registers
    if (!(temperature == temperature) || !(cfg_scale == cfg_scale) || isinf(temperature) || isinf(cfg_scale))
        return HAWK_ERR_PARAM;
    if (!(temperature > 0.f)) return HAWK_ERR_PARAM;
    if (!hawk_host::aligned16(logits) || !hawk_host::aligned16(q_probs) || (p_debug && !hawk_host::aligned16(p_debug)))
        return HAWK_ERR_ALIGN;
    const size_t need = hawk_cfg_accept_workspace_bytes(B, K, V);
    if (!workspace || workspace_bytes < need) return HAWK_ERR_WORKSPACE;
    if (!hawk_host::aligned16(workspace)) return HAWK_ERR_ALIGN;
    return HAWK_OK;
}

namespace {
hawk_status cfg_accept_impl(const float *logits, int guided_in, const float *q_probs, const int32_t *draft,
                            const float *u_accept, const float *u_resample, int B, int K, int V, int v_begin,
                            int v_end, float cfg_scale, float temperature, int top_k, int has_bonus_row,
                            int32_t *accept_len, int32_t *out_token, float *p_debug, void *workspace,
                            size_t workspace_bytes, int32_t *dev_status, hawk_stream_t stream)
{
    const hawk_status chk = hawk_host::check_cfg_accept_args(logits, q_probs, draft, u_accept, u_resample, B, K, V, v_begin,
                                                            v_end, cfg_scale, temperature, accept_len, out_token, p_debug,
                                                            workspace, workspace_bytes);
    if (chk != HAWK_OK) return chk;
    if (B == 0) return HAWK_OK;
    const int n = v_end - v_begin;
    if (!hawk_host::is_sm100(nullptr)) return HAWK_ERR_UNSUPPORTED;

    AcceptParams P;
    P.logits = logits;
    P.q = q_probs;
    P.draft = draft;
    P.u_acc = u_accept;
    P.u_res = u_resample;
    P.B = B;
    P.K = K;
    P.rows = K + (has_bonus_row ? 1 : 0);
    P.V = V;
    P.v_begin = v_begin;
    P.n = n;
    P.cfg_scale = cfg_scale;
    P.temperature = temperature;
    P.top_k = top_k;
    P.vec_ok = (V % 4 == 0 && v_begin % 4 == 0) ? 1 : 0;
    P.guided_in = guided_in;
    P.row_out = static_cast<int32_t *>(workspace);
    P.p_debug = p_debug;
    P.dev_status = dev_status;

    cudaStream_t st = reinterpret_cast<cudaStream_t>(stream);
    const int grid = B * P.rows;
    cudaError_t err;
    // more rows than SMs: the later rows can see the verdicts of the earlier ones (see accept_rows_kernel)
    int sm_count = 0;
    (void)hawk_host::is_sm100(&sm_count);
#ifndef HAWK_ACCEPT_SKIP_WAVES_X4
#define HAWK_ACCEPT_SKIP_WAVES_X4 6  // quarter waves of rows from which verdicts are marked and looked at: 6 = 1.5 waves
#endif
    P.skip_mode = (4 * grid > HAWK_ACCEPT_SKIP_WAVES_X4 * sm_count && !p_debug) ? 1 : 0;
    if (P.skip_mode) {
        err = hawk_host::launch_dependent(accept_clear_kernel, dim3((grid + 255) / 256), dim3(256), 0, st, P.row_out, grid);
        if (err != cudaSuccess) return HAWK_ERR_CUDA;
    }
    // 16 ids per thread; the block as wide as the row needs
    if (n <= 4096) err = launch_rows<256, 4>(P, grid, st);
    else if (n <= 8192) err = launch_rows<512, 4>(P, grid, st);
    else if (n <= 16384) err = launch_rows<1024, 4>(P, grid, st);
    else err = launch_rows<1024, 8>(P, grid, st);
    if (err != cudaSuccess) return HAWK_ERR_CUDA;
    err = hawk_host::launch_dependent(accept_finalize_kernel, dim3((B + 127) / 128), dim3(128), 0, st,
                                      static_cast<const int32_t *>(P.row_out), B, K, P.rows, accept_len, out_token);
    return err == cudaSuccess ? HAWK_OK : HAWK_ERR_CUDA;
}
}  // namespace

extern "C" hawk_status hawk_cfg_accept(const float *logits, const float *q_probs, const int32_t *draft,
                                       const float *u_accept, const float *u_resample, int B, int K, int V,
                                       int v_begin, int v_end, float cfg_scale, float temperature, int top_k,
                                       int has_bonus_row, int32_t *accept_len, int32_t *out_token, float *p_debug,
                                       void *workspace, size_t workspace_bytes, int32_t *dev_status,
                                       hawk_stream_t stream)
{
    const hawk_host::NvtxRange nvtx_range("hawk_cfg_accept");
    return cfg_accept_impl(logits, 0, q_probs, draft, u_accept, u_resample, B, K, V, v_begin, v_end, cfg_scale,
                           temperature, top_k, has_bonus_row, accept_len, out_token, p_debug, workspace,
                           workspace_bytes, dev_status, stream);
}

extern "C" hawk_status hawk_cfg_accept_guided(const float *guided, const float *q_probs, const int32_t *draft,
                                              const float *u_accept, const float *u_resample, int B, int K, int V,
                                              int v_begin, int v_end, int top_k, int has_bonus_row,
                                              int32_t *accept_len, int32_t *out_token, float *p_debug,
                                              void *workspace, size_t workspace_bytes, int32_t *dev_status,
                                              hawk_stream_t stream)
{
    const hawk_host::NvtxRange nvtx_range("hawk_cfg_accept_guided");
    return cfg_accept_impl(guided, 1, q_probs, draft, u_accept, u_resample, B, K, V, v_begin, v_end, 1.0f, 1.0f, top_k,
                           has_bonus_row, accept_len, out_token, p_debug, workspace, workspace_bytes, dev_status,
                           stream);
}


extern "C" size_t hawk_tree_accept_workspace_bytes(int B, int N)
{
    if (B <= 0 || N <= 0) return 0;
    return (static_cast<size_t>(B) + 1) * static_cast<size_t>(N) * sizeof(int32_t);  // verdicts, then a parent per node
}

namespace {
hawk_status tree_accept_impl(const float *logits, int guided_in, const float *q_probs, const int32_t *node_token,
                             const int32_t *node_q, const int32_t *child_begin, const float *u_accept,
                             const float *u_resample, int B, int N, int NQ, int V, int v_begin, int v_end,
                             float cfg_scale, float temperature, int top_k, int max_depth, int32_t *accept_len,
                             int32_t *out_token, int32_t *path, void *workspace, size_t workspace_bytes,
                             int32_t *dev_status, hawk_stream_t stream)
{
    if (B < 0 || N < 0 || NQ < 0 || V < 0 || max_depth < 0) return HAWK_ERR_SHAPE;
    if (B == 0) return HAWK_OK;
    if (!logits || !q_probs || !node_token || !node_q || !child_begin || !u_accept || !u_resample || !accept_len ||
        !out_token)
        return HAWK_ERR_NULL;
    if (N < 1 || NQ < 1) return HAWK_ERR_SHAPE;
    if (v_begin < 0 || v_end > V || v_begin >= v_end) return HAWK_ERR_SHAPE;
    if (N > 65536) return HAWK_ERR_UNSUPPORTED;
    const int n = v_end - v_begin;
    if (n > 32768) return HAWK_ERR_UNSUPPORTED;  // one row must fit one block's registers
    if (!(temperature == temperature) || !(cfg_scale == cfg_scale) || isinf(temperature) || isinf(cfg_scale))
        return HAWK_ERR_PARAM;
    if (!(temperature > 0.f)) return HAWK_ERR_PARAM;
    if (!hawk_host::aligned16(logits) || !hawk_host::aligned16(q_probs)) return HAWK_ERR_ALIGN;
    const size_t need = hawk_tree_accept_workspace_bytes(B, N);
    if (!workspace || workspace_bytes < need) return HAWK_ERR_WORKSPACE;
    if (!hawk_host::aligned16(workspace)) return HAWK_ERR_ALIGN;
    if (!hawk_host::is_sm100(nullptr)) return HAWK_ERR_UNSUPPORTED;

    TreeParams P;
    P.logits = logits;
    P.q = q_probs;
    P.node_token = node_token;
    P.node_q = node_q;
    P.child_begin = child_begin;
    P.u_acc = u_accept;
    P.u_res = u_resample;
    P.B = B;
    P.N = N;
    P.NQ = NQ;
    P.V = V;
    P.v_begin = v_begin;
    P.n = n;
    P.cfg_scale = cfg_scale;
    P.temperature = temperature;
    P.top_k = top_k;
    P.vec_ok = (V % 4 == 0 && v_begin % 4 == 0) ? 1 : 0;
    P.guided_in = guided_in;
    P.verdict = static_cast<int32_t *>(workspace);
    int32_t *parent = P.verdict + static_cast<size_t>(B) * N;
    P.parent = parent;
    P.dev_status = dev_status;

    cudaStream_t st = reinterpret_cast<cudaStream_t>(stream);
    const int grid = B * N;
    cudaError_t err;
    int sm_count = 0;
    (void)hawk_host::is_sm100(&sm_count);
    P.skip_mode = grid > sm_count + sm_count / 2 ? 1 : 0;  // as in the chain: worth it from 1.5 waves on
    if (P.skip_mode) {
        err = hawk_host::launch_dependent(tree_prepare_kernel, dim3((grid + 255) / 256), dim3(256), 0, st, P.verdict, parent,
                                          child_begin, B, N);
        if (err != cudaSuccess) return HAWK_ERR_CUDA;
    }
    if (n <= 4096) err = launch_tree_rows<256, 4>(P, grid, st);
    else if (n <= 8192) err = launch_tree_rows<512, 4>(P, grid, st);
    else if (n <= 16384) err = launch_tree_rows<1024, 4>(P, grid, st);
    else err = launch_tree_rows<1024, 8>(P, grid, st);
    if (err != cudaSuccess) return HAWK_ERR_CUDA;
    err = hawk_host::launch_dependent(tree_walk_kernel, dim3((B + 127) / 128), dim3(128), 0, st,
                                      static_cast<const int32_t *>(P.verdict), B, N, path ? max_depth : 0, accept_len,
                                      out_token, path, dev_status);
    return err == cudaSuccess ? HAWK_OK : HAWK_ERR_CUDA;
}
}  // namespace

extern "C" hawk_status hawk_tree_accept(const float *logits, const float *q_probs, const int32_t *node_token,
                                        const int32_t *node_q, const int32_t *child_begin, const float *u_accept,
                                        const float *u_resample, int B, int N, int NQ, int V, int v_begin,
                                        int v_end, float cfg_scale, float temperature, int top_k, int max_depth,
                                        int32_t *accept_len, int32_t *out_token, int32_t *path, void *workspace,
                                        size_t workspace_bytes, int32_t *dev_status, hawk_stream_t stream)
{
    const hawk_host::NvtxRange nvtx_range("hawk_tree_accept");
    return tree_accept_impl(logits, 0, q_probs, node_token, node_q, child_begin, u_accept, u_resample, B, N, NQ, V,
                            v_begin, v_end, cfg_scale, temperature, top_k, max_depth, accept_len, out_token, path,
                            workspace, workspace_bytes, dev_status, stream);
}

extern "C" hawk_status hawk_tree_accept_guided(const float *guided, const float *q_probs, const int32_t *node_token,
                                               const int32_t *node_q, const int32_t *child_begin,
                                               const float *u_accept, const float *u_resample, int B, int N, int NQ,
                                               int V, int v_begin, int v_end, int top_k, int max_depth,
                                               int32_t *accept_len, int32_t *out_token, int32_t *path,
                                               void *workspace, size_t workspace_bytes, int32_t *dev_status,
                                               hawk_stream_t stream)
{
    const hawk_host::NvtxRange nvtx_range("hawk_tree_accept_guided");
    return tree_accept_impl(guided, 1, q_probs, node_token, node_q, child_begin, u_accept, u_resample, B, N, NQ, V,
                            v_begin, v_end, 1.0f, 1.0f, top_k, max_depth, accept_len, out_token, path, workspace,
                            workspace_bytes, dev_status, stream);
}


extern "C" size_t hawk_pool_sample_workspace_bytes(int B, int NQ)
{
    if (B <= 0 || NQ <= 0) return 0;
    return static_cast<size_t>(B) * static_cast<size_t>(NQ) * sizeof(int32_t);
}

extern "C" hawk_status hawk_pool_sample(const float *pool_q, const float *u, const int32_t *node_q,
                                        int32_t *node_token, int B, int NQ, int N, int V, int v_begin, int v_end,
                                        void *workspace, size_t workspace_bytes, int32_t *dev_status,
                                        hawk_stream_t stream)
{
    const hawk_host::NvtxRange nvtx_range("hawk_pool_sample");
    if (B < 0 || NQ < 0 || N < 0 || V < 0) return HAWK_ERR_SHAPE;
    if (B == 0) return HAWK_OK;
    if (!pool_q || !u || !node_q || !node_token) return HAWK_ERR_NULL;
    if (NQ < 1 || N < 1 || v_begin < 0 || v_end > V || v_begin >= v_end) return HAWK_ERR_SHAPE;
    const int n = v_end - v_begin;
    if (n > 32768) return HAWK_ERR_UNSUPPORTED;
    if (!hawk_host::aligned16(pool_q)) return HAWK_ERR_ALIGN;
    const size_t need = hawk_pool_sample_workspace_bytes(B, NQ);
    if (!workspace || workspace_bytes < need) return HAWK_ERR_WORKSPACE;
    if (!hawk_host::aligned16(workspace)) return HAWK_ERR_ALIGN;
    if (!hawk_host::is_sm100(nullptr)) return HAWK_ERR_UNSUPPORTED;
    cudaStream_t st = reinterpret_cast<cudaStream_t>(stream);
    const int vec_ok = (V % 4 == 0 && v_begin % 4 == 0) ? 1 : 0;
    const int grid = B * NQ;
    cudaError_t err;
    if (n <= 4096)
        err = hawk_host::launch_dependent(pool_sample_kernel<256, 4>, dim3(grid), dim3(256), 0, st, pool_q, u, node_q,
                                          node_token, NQ, N, V, v_begin, n, vec_ok, dev_status);
    else if (n <= 8192)
        err = hawk_host::launch_dependent(pool_sample_kernel<512, 4>, dim3(grid), dim3(512), 0, st, pool_q, u, node_q,
                                          node_token, NQ, N, V, v_begin, n, vec_ok, dev_status);
    else if (n <= 16384)
        err = hawk_host::launch_dependent(pool_sample_kernel<1024, 4>, dim3(grid), dim3(1024), 0, st, pool_q, u, node_q,
                                          node_token, NQ, N, V, v_begin, n, vec_ok, dev_status);
    else
        err = hawk_host::launch_dependent(pool_sample_kernel<1024, 8>, dim3(grid), dim3(1024), 0, st, pool_q, u, node_q,
                                          node_token, NQ, N, V, v_begin, n, vec_ok, dev_status);
    return err == cudaSuccess ? HAWK_OK : HAWK_ERR_CUDA;
}

// ------------------------------------------------------------------------------------------------
// hawk_cfg_accept_noalloc: the same verification for callers that have no device memory to lend
// as a workspace.  The per-row verdicts go to a fixed array that lives in the library's own
// device image instead.
namespace {

constexpr int kBuiltinRows = 16384;  // verdict slots: B * (K + 1) must not exceed this (64 KiB)
static __device__ __align__(256) int32_t g_builtin_row_out[kBuiltinRows];

constexpr int kMaxDevices = 64;
std::mutex g_builtin_mutex;
void *g_builtin_addr[kMaxDevices];  // device address of the array, per device, once looked up

// The array's name is only a host-side handle; kernels need its device address, which differs per
// device.  Looked up once per device, with that device current.
hawk_status builtin_scratch(void **ptr)
{
    int dev = -1;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= kMaxDevices) return HAWK_ERR_CUDA;
    std::lock_guard<std::mutex> lock(g_builtin_mutex);
    if (!g_builtin_addr[dev]) {
        void *p = nullptr;
        if (cudaGetSymbolAddress(&p, g_builtin_row_out) != cudaSuccess || !p) return HAWK_ERR_CUDA;
        g_builtin_addr[dev] = p;
    }
    *ptr = g_builtin_addr[dev];
    return HAWK_OK;
}

}  // namespace

extern "C" size_t hawk_cfg_accept_noalloc_max_rows(void) { return kBuiltinRows; }

extern "C" hawk_status hawk_cfg_accept_noalloc(const float *logits, const float *q_probs, const int32_t *draft,
                                               const float *u_accept, const float *u_resample, int B, int K, int V,
                                               int v_begin, int v_end, float cfg_scale, float temperature,
                                               int top_k, int has_bonus_row, int32_t *accept_len,
                                               int32_t *out_token, int32_t *dev_status, hawk_stream_t stream)
{
    const hawk_host::NvtxRange nvtx_range("hawk_cfg_accept_noalloc");
    if (B < 0 || K < 0 || V < 0) return HAWK_ERR_SHAPE;
    if (B == 0) return HAWK_OK;
    if (K < 1 || K > 16) return HAWK_ERR_UNSUPPORTED;
    if (static_cast<long long>(B) * (K + 1) > kBuiltinRows) return HAWK_ERR_WORKSPACE;  // beyond the built-in array
    void *scratch = nullptr;
    const hawk_status rc = builtin_scratch(&scratch);
    if (rc != HAWK_OK) return rc;
    // Every row of the step writes its own slot before the per-sequence pass reads it, so the array
    // needs no clearing even though it still holds the previous call's verdicts.
    return hawk_cfg_accept(logits, q_probs, draft, u_accept, u_resample, B, K, V, v_begin, v_end, cfg_scale,
                           temperature, top_k, has_bonus_row, accept_len, out_token, nullptr, scratch,
                           sizeof(int32_t) * kBuiltinRows, dev_status, stream);
}
