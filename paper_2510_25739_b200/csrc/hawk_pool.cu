// Speculation cache and spatial sampling pool (Sec. 4.2, "Dual Direction Drafting Heads" and
// "Spatial Sampling Pool", Eqs. 1-5): the step that feeds the verification with candidates.
//
// The vertical draft head of depth d, run at raster position P, predicts the token at P + IW * d
// (IW tokens per image row).  That prediction is of no use until decoding reaches the target row, so it
// is kept in a cache of IW * VSD * (VSD + 1) / 2 slots per sequence (Eq. 2): for a column and a depth
// d there are never more than d predictions alive, one per source row modulo d.  When position
// T + n is speculated, its pool is the horizontal head's distribution for T + n plus, for every
// dv = 1 .. VSD, the cached prediction made dv rows above with depth dv (Eqs. 3-5).  A slot carries the
// position that wrote it, so a prediction that was never made (no step started at that position) is
// recognised and replaced by a second draw from the horizontal distribution.
//
// Everything here is index arithmetic and row copies; the one numerical kernel, drawing a candidate
// token from every pool distribution by inverse CDF, lives with the accept kernels (hawk_accept.cu).
#include "hawk_common.cuh"

namespace {

__host__ __device__ __forceinline__ int tri(int m) { return m * (m + 1) / 2; }

// Slot of the prediction made at raster position `pos` by the vertical head of depth d (1-based).
__host__ __device__ __forceinline__ int cache_slot(int IW, int VSD, int pos, int d)
{
    const int col = pos % IW, row = pos / IW;
    return col * tri(VSD) + tri(d - 1) + row % d;
}

// Copies n floats; both rows 16-byte aligned when vec is set.
__device__ __forceinline__ void copy_row(float *dst, const float *src, int n, bool vec)
{
    if (vec) {
        const float4 *s4 = reinterpret_cast<const float4 *>(src);
        float4 *d4 = reinterpret_cast<float4 *>(dst);
        for (int i = blockIdx.y * blockDim.x + threadIdx.x; i < n / 4; i += gridDim.y * blockDim.x) d4[i] = s4[i];
    } else {
        for (int i = blockIdx.y * blockDim.x + threadIdx.x; i < n; i += gridDim.y * blockDim.x) dst[i] = src[i];
    }
}

// blockIdx.x = b * VSD + (d - 1): stores the depth-d prediction of sequence b.
__global__ void cache_put_kernel(const float *q_vert, const int32_t *position, float *rows, int32_t *tags, int IW,
                                 int VSD, int V, int slots, int vec)
{
    hawk::allow_dependent_launch();
    hawk::grid_dependency_wait();
    const int b = blockIdx.x / VSD, d = blockIdx.x % VSD + 1;
    const int pos = position[b];
    if (pos < 0) return;
    const int slot = cache_slot(IW, VSD, pos, d);
    if (!HAWK_IN_BOUNDS(nullptr, slot, slots)) return;  // (debug build; these kernels have no status word: the copy is skipped)
    copy_row(rows + (static_cast<size_t>(b) * slots + slot) * V, q_vert + (static_cast<size_t>(b) * VSD + d - 1) * V, V,
             vec != 0);
    if (blockIdx.y == 0 && threadIdx.x == 0) tags[b * slots + slot] = pos;
}

// blockIdx.x = (b * K + n - 1) * (1 + VSD) + j: pool row j of speculation offset n of sequence b.
// j = 0: the horizontal head's distribution for T + n; j = dv >= 1: the cached vertical prediction made
// dv rows above T + n with depth dv, or the horizontal distribution again if that prediction is missing.
__global__ void pool_build_kernel(const float *q_horiz, const float *rows, const int32_t *tags, const int32_t *position,
                                  float *pool_q, int32_t *pool_source, int K, int IW, int VSD, int V, int slots, int vec)
{
    hawk::allow_dependent_launch();
    hawk::grid_dependency_wait();
    const int width = 1 + VSD;
    const int j = blockIdx.x % width, bn = blockIdx.x / width;
    const int n = bn % K + 1, b = bn / K;
    const float *src = q_horiz + (static_cast<size_t>(b) * K + n - 1) * V;
    int source = 0;
    if (j > 0) {
        const int target = position[b] + n, from = target - IW * j;
        source = -j;  // missing until found
        if (position[b] >= 0 && from >= 0) {
            const int slot = cache_slot(IW, VSD, from, j);
            if (HAWK_IN_BOUNDS(nullptr, slot, slots) && tags[b * slots + slot] == from) {
                src = rows + (static_cast<size_t>(b) * slots + slot) * V;
                source = j;
            }
        }
    }
    copy_row(pool_q + static_cast<size_t>(blockIdx.x) * V, src, V, vec != 0);
    if (pool_source && blockIdx.y == 0 && threadIdx.x == 0) pool_source[blockIdx.x] = source;
}

}  // namespace

extern "C" int hawk_spec_cache_slots(int IW, int VSD)
{
    if (IW < 1 || VSD < 1) return 0;
    return IW * tri(VSD);
}

extern "C" int hawk_spec_cache_slot(int IW, int VSD, int position, int depth)
{
    if (IW < 1 || VSD < 1 || position < 0 || depth < 1 || depth > VSD) return -1;
    return cache_slot(IW, VSD, position, depth);
}

extern "C" hawk_status hawk_spec_cache_clear(int32_t *cache_tags, int B, int IW, int VSD, hawk_stream_t stream)
{
    const hawk_host::NvtxRange nvtx_range("hawk_spec_cache_clear");
    if (B < 0 || IW < 1 || VSD < 1) return HAWK_ERR_SHAPE;
    if (B == 0) return HAWK_OK;
    if (!cache_tags) return HAWK_ERR_NULL;
    const size_t bytes = static_cast<size_t>(B) * hawk_spec_cache_slots(IW, VSD) * sizeof(int32_t);
    return cudaMemsetAsync(cache_tags, 0xFF, bytes, reinterpret_cast<cudaStream_t>(stream)) == cudaSuccess
               ? HAWK_OK
               : HAWK_ERR_CUDA;  // every tag -1: no prediction stored
}

extern "C" hawk_status hawk_spec_cache_put(const float *q_vert, const int32_t *position, float *cache_rows,
                                           int32_t *cache_tags, int B, int IW, int VSD, int V, hawk_stream_t stream)
{
    const hawk_host::NvtxRange nvtx_range("hawk_spec_cache_put");
    if (B < 0 || IW < 1 || VSD < 1 || V < 1) return HAWK_ERR_SHAPE;
    if (B == 0) return HAWK_OK;
    if (!q_vert || !position || !cache_rows || !cache_tags) return HAWK_ERR_NULL;
    if (VSD > 8) return HAWK_ERR_UNSUPPORTED;
    if (!hawk_host::is_sm100(nullptr)) return HAWK_ERR_UNSUPPORTED;
    const int vec = (V % 4 == 0 && hawk_host::aligned16(q_vert) && hawk_host::aligned16(cache_rows)) ? 1 : 0;
    const int chunks = (V + 4 * 256 * 4 - 1) / (4 * 256 * 4);  // 16 elements per thread
    const cudaError_t err = hawk_host::launch_dependent(cache_put_kernel, dim3(B * VSD, chunks), dim3(256), 0,
                                                        reinterpret_cast<cudaStream_t>(stream), q_vert, position,
                                                        cache_rows, cache_tags, IW, VSD, V,
                                                        hawk_spec_cache_slots(IW, VSD), vec);
    return err == cudaSuccess ? HAWK_OK : HAWK_ERR_CUDA;
}

extern "C" hawk_status hawk_pool_build(const float *q_horiz, const float *cache_rows, const int32_t *cache_tags,
                                       const int32_t *position, float *pool_q, int32_t *pool_source, int B, int K,
                                       int IW, int VSD, int V, hawk_stream_t stream)
{
    const hawk_host::NvtxRange nvtx_range("hawk_pool_build");
    if (B < 0 || K < 0 || IW < 1 || VSD < 1 || V < 1) return HAWK_ERR_SHAPE;
    if (B == 0 || K == 0) return HAWK_OK;
    if (!q_horiz || !cache_rows || !cache_tags || !position || !pool_q) return HAWK_ERR_NULL;
    if (VSD > 8 || static_cast<long long>(B) * K * (1 + VSD) >= (1ll << 31)) return HAWK_ERR_UNSUPPORTED;
    if (!hawk_host::is_sm100(nullptr)) return HAWK_ERR_UNSUPPORTED;
    const int vec = (V % 4 == 0 && hawk_host::aligned16(q_horiz) && hawk_host::aligned16(cache_rows) &&
                     hawk_host::aligned16(pool_q))
                        ? 1
                        : 0;
    const int chunks = (V + 4 * 256 * 4 - 1) / (4 * 256 * 4);
    const cudaError_t err = hawk_host::launch_dependent(pool_build_kernel, dim3(B * K * (1 + VSD), chunks), dim3(256), 0,
                                                        reinterpret_cast<cudaStream_t>(stream), q_horiz, cache_rows,
                                                        cache_tags, position, pool_q, pool_source, K, IW, VSD, V,
                                                        hawk_spec_cache_slots(IW, VSD), vec);
    return err == cudaSuccess ? HAWK_OK : HAWK_ERR_CUDA;
}
