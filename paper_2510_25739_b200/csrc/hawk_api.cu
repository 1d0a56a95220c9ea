// Library-wide entry points (status strings, version) and host helpers shared by the launchers.
#include <cudaTypedefs.h>

#include <mutex>

#include "hawk_common.cuh"

extern "C" const char *hawk_status_string(hawk_status status)
{
    switch (status) {
        case HAWK_OK: return "ok";
        case HAWK_ERR_NULL: return "a required pointer is NULL";
        case HAWK_ERR_SHAPE: return "sizes are negative or contradict each other";
        case HAWK_ERR_ALIGN: return "a tensor base is not 16-byte aligned";
        case HAWK_ERR_UNSUPPORTED: return "value outside what the sm_100a kernels support";
        case HAWK_ERR_WORKSPACE: return "workspace missing or too small";
        case HAWK_ERR_PARAM: return "a scalar parameter is not a usable number";
        case HAWK_ERR_CUDA: return "the CUDA runtime or driver refused a call";
    }
    return "unknown status";
}

extern "C" int hawk_version(void) { return HAWK_VERSION_NUMBER; }

namespace hawk_host {

static PFN_cuTensorMapEncodeTiled_v12000 encode_fn()
{
    static PFN_cuTensorMapEncodeTiled_v12000 fn = nullptr;
    static std::once_flag once;
    std::call_once(once, [] {
        void *p = nullptr;
        cudaDriverEntryPointQueryResult qres;
        if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &p, cudaEnableDefault, &qres) == cudaSuccess &&
            qres == cudaDriverEntryPointSuccess)
            fn = reinterpret_cast<PFN_cuTensorMapEncodeTiled_v12000>(p);
    });
    return fn;
}

bool encode_bf16_rows_sw128(CUtensorMap *map, const void *base, uint64_t rows, uint64_t cols, uint32_t box_rows,
                            bool promote_l2_256)
{
    PFN_cuTensorMapEncodeTiled_v12000 fn = encode_fn();
    if (!fn) return false;
    cuuint64_t dims[2] = {cols, rows};
    cuuint64_t strides[1] = {cols * 2};  // bytes between rows
    cuuint32_t box[2] = {64, box_rows};  // 64 bf16 = 128 bytes = one swizzle span
    cuuint32_t estr[2] = {1, 1};
    CUresult r = fn(map, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, const_cast<void *>(base), dims, strides, box, estr,
                    CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B,
                    promote_l2_256 ? CU_TENSOR_MAP_L2_PROMOTION_L2_256B : CU_TENSOR_MAP_L2_PROMOTION_L2_128B,
                    CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
    return r == CUDA_SUCCESS;
}

bool is_sm100(int *sm_count)
{
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess) return false;
    int major = 0, sms = 0;
    if (cudaDeviceGetAttribute(&major, cudaDevAttrComputeCapabilityMajor, dev) != cudaSuccess) return false;
    if (cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess) return false;
    if (sm_count) *sm_count = sms;
    return major == 10;
}

}  // namespace hawk_host
