// Host-side support shared by the tensor-core kernels: the device status word that a kernel sets
// when one of its bounded waits runs out, the wait limit, per-device launch bookkeeping, and the
// tensor-map encoder for packed operands.
#include <atomic>
#include <mutex>
#include <set>

#include "bnn_common.cuh"
#include "tcgen05.cuh"

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

// ---- per-device bookkeeping -------------------------------------------------------------
// A process may drive several devices: the status word's address, the SM count and the kernels
// whose dynamic shared-memory limit has been raised are kept per device ordinal.
namespace {

constexpr int kMaxDevices = 64;
struct DeviceInfo {
    bool looked_up = false;
    int sms = 0;
    int* status = nullptr;
    std::set<const void*> raised;    // kernels with cudaFuncAttributeMaxDynamicSharedMemorySize set
};
std::mutex g_mutex;
DeviceInfo g_devices[kMaxDevices];
std::atomic<long long> g_wait_limit_clocks{2000000000LL};   // about a second of SM clocks

// Entry of the current device (g_mutex held), or nullptr.
DeviceInfo* current_device() {
    int dev = -1;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= kMaxDevices) return nullptr;
    DeviceInfo& d = g_devices[dev];
    if (!d.looked_up) {
        void* p = nullptr;
        if (cudaDeviceGetAttribute(&d.sms, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess ||
            cudaGetSymbolAddress(&p, g_tc_status) != cudaSuccess)
            return nullptr;
        d.status = static_cast<int*>(p);
        d.looked_up = true;
    }
    return &d;
}

}  // namespace

int device_sm_count() {
    std::lock_guard<std::mutex> lock(g_mutex);
    DeviceInfo* d = current_device();
    return d ? d->sms : 0;
}

bool ensure_dynamic_smem(const void* kernel, int bytes) {
    std::lock_guard<std::mutex> lock(g_mutex);
    DeviceInfo* d = current_device();
    if (!d) return false;
    if (d->raised.count(kernel)) return true;
    if (cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, bytes) != cudaSuccess) return false;
    d->raised.insert(kernel);
    return true;
}

tc::TcStatus tc_status() {
    std::lock_guard<std::mutex> lock(g_mutex);
    DeviceInfo* d = current_device();
    return tc::TcStatus{d ? d->status : nullptr, g_wait_limit_clocks.load()};
}

long long set_wait_limit_clocks(long long clocks) { return g_wait_limit_clocks.exchange(clocks); }

int read_tc_status(int* out) {
    return cudaMemcpyFromSymbol(out, g_tc_status, sizeof(int)) == cudaSuccess ? BNN_OK : BNN_ERR_CUDA;
}

int copy_tc_status_async(int* dst, cudaStream_t st) {
    const tc::TcStatus s = tc_status();
    if (!s.word) return BNN_ERR_CUDA;
    return cudaMemcpyAsync(dst, s.word, sizeof(int), cudaMemcpyDefault, st) == cudaSuccess ? BNN_OK : BNN_ERR_CUDA;
}

int reset_tc_status_async(cudaStream_t st) {
    const tc::TcStatus s = tc_status();
    if (!s.word) return BNN_ERR_CUDA;
    return cudaMemsetAsync(s.word, 0, sizeof(int), st) == cudaSuccess ? BNN_OK : BNN_ERR_CUDA;
}

// ---- a launch whose wait runs out ----------------------------------------------------------
// One CTA, one warp: it waits on an mbarrier on which nothing ever arrives.  The wait gives up
// after the limit, the kernel sets the status word and returns like every tensor-core kernel
// does in that case.  It exists so that the give-up path can be exercised without a fault.
namespace {
__global__ void wait_probe_kernel(tc::TcStatus status) {
    __shared__ uint64_t bar;
    __shared__ tc::WaitState wait;
    if (threadIdx.x == 0) {
        tc::mbar_init(tc::smem_u32(&bar), 1);
        tc::wait_state_init(&wait, status);
        tc::mbar_init_fence();
    }
    __syncthreads();
    const bool ok = tc::warp_wait(tc::smem_u32(&bar), 0u, &wait.abort, threadIdx.x & 31);
    if (threadIdx.x == 0 && !ok) atomicExch(status.word, 1);
}
}  // namespace

int launch_wait_probe(cudaStream_t st) {
    const tc::TcStatus s = tc_status();
    if (!s.word) return BNN_ERR_CUDA;
    wait_probe_kernel<<<1, 32, 0, st>>>(s);
    return launch_status();
}

}  // namespace bnn
