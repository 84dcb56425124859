// Host-side support shared by the tensor-core kernels: the device status word that a kernel sets
// when one of its bounded waits runs out, and the tensor-map encoder for packed operands.
#include "bnn_common.cuh"

namespace bnn {

__device__ int g_tc_status = 0;  // set to 1 by a CTA whose bounded wait ran out

// The driver's tensor-map encoder is looked up through the runtime, so that the library does not
// link against the driver library (which only exists on machines with a GPU).
bool encode_packed_map(CUtensorMap* map, const uint32_t* base, int ld, int rows, int K, int box_rows) {
    using EncodeFn = CUresult (*)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*,
                                  const cuuint64_t*, const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave,
                                  CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);
    static EncodeFn encode = nullptr;
    if (!encode) {
        void* fn = nullptr;
        cudaDriverEntryPointQueryResult res;
        if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &fn, cudaEnableDefault, &res) != cudaSuccess ||
            res != cudaDriverEntryPointSuccess || !fn)
            return false;
        encode = reinterpret_cast<EncodeFn>(fn);
    }
    const cuuint64_t dims[2] = {(cuuint64_t)words_for(K), (cuuint64_t)rows};
    const cuuint64_t strides[1] = {(cuuint64_t)ld * sizeof(uint32_t)};   // bytes between rows (multiple of 16)
    const cuuint32_t box[2] = {16u, (cuuint32_t)box_rows};
    const cuuint32_t estr[2] = {1u, 1u};
    return encode(map, CU_TENSOR_MAP_DATA_TYPE_UINT32, 2, const_cast<uint32_t*>(base), dims, strides, box, estr,
                  CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_64B, CU_TENSOR_MAP_L2_PROMOTION_L2_128B,
                  CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

// Device address of the status word (one per device would need a table; one device is used).
int* tc_status_ptr() {
    static int* ptr = nullptr;
    if (!ptr && cudaGetSymbolAddress(reinterpret_cast<void**>(&ptr), g_tc_status) != cudaSuccess) ptr = nullptr;
    return ptr;
}

int read_tc_status(int* out) {
    return cudaMemcpyFromSymbol(out, g_tc_status, sizeof(int)) == cudaSuccess ? BNN_OK : BNN_ERR_CUDA;
}

}  // namespace bnn
