// Host utilities: tensor-map encoding through the runtime's driver entry point lookup, device
// queries, and the fp32 -> bf16 pre-pass used for RPX_F32 inputs.
#include <cuda_bf16.h>

#include <atomic>
#include <mutex>

#include "rpx_internal.h"
#include "rpx_ptx.cuh"

namespace rpx {

namespace {

typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*,
                                  const cuuint64_t*, const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave,
                                  CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

EncodeTiledFn encode_fn() {
    static EncodeTiledFn fn = nullptr;
    static std::once_flag once;
    std::call_once(once, [] {
        void* p = nullptr;
        cudaDriverEntryPointQueryResult q;
        if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &p, cudaEnableDefault, &q) == cudaSuccess &&
            q == cudaDriverEntryPointSuccess)
            fn = reinterpret_cast<EncodeTiledFn>(p);
    });
    return fn;
}

__global__ void cast_f32_bf16_kernel(const float* __restrict__ src, int64_t src_row_stride,
                                     __nv_bfloat16* __restrict__ dst, int64_t rows, int64_t cols) {
    const int64_t total = rows * cols;
    for (int64_t i = blockIdx.x * static_cast<int64_t>(blockDim.x) + threadIdx.x; i < total;
         i += static_cast<int64_t>(gridDim.x) * blockDim.x) {
        const int64_t r = i / cols, c = i - r * cols;
        dst[i] = __float2bfloat16_rn(src[r * src_row_stride + c]);
    }
}

// One thread waits on an mbarrier nobody arrives on, so the bounded wait has to run out.
__global__ void bounded_wait_selftest_kernel(long long limit_cycles, int32_t* status) {
    __shared__ uint64_t bar;
    __shared__ uint32_t abort_flag;
    if (threadIdx.x == 0) {
        mbar_init(&bar, 1);
        abort_flag = 0;
        fence_barrier_init();
    }
    __syncthreads();
    if (threadIdx.x == 0) {
        const bool completed = mbar_wait(&bar, 0, &abort_flag, limit_cycles);
        if (!completed && abort_flag != 0u && status != nullptr) atomicCAS(status, 0, RPX_ERR_TIMEOUT);
    }
}

}  // namespace

rpx_status_t launch_bounded_wait_selftest(long long limit_cycles, int32_t* status, cudaStream_t stream) {
    bounded_wait_selftest_kernel<<<1, 32, 0, stream>>>(limit_cycles, status);
    return cudaGetLastError() == cudaSuccess ? RPX_OK : RPX_ERR_CUDA;
}

rpx_status_t encode_tmap_bf16(CUtensorMap* map, const void* base, int rank, const uint64_t* dims,
                              const uint64_t* strides_bytes, const uint32_t* box) {
    EncodeTiledFn fn = encode_fn();
    if (!fn) return RPX_ERR_CUDA;
    cuuint64_t gdim[5], gstride[4];
    cuuint32_t bdim[5], estride[5];
    for (int i = 0; i < rank; ++i) {
        gdim[i] = dims[i];
        bdim[i] = box[i];
        estride[i] = 1;
        if (i + 1 < rank) gstride[i] = strides_bytes[i];
    }
    const CUresult rc = fn(map, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, static_cast<cuuint32_t>(rank), const_cast<void*>(base),
                           gdim, gstride, bdim, estride, CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B,
                           CU_TENSOR_MAP_L2_PROMOTION_L2_256B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
    return rc == CUDA_SUCCESS ? RPX_OK : RPX_ERR_CUDA;
}

int sm_count() {
    int dev = 0, n = 0;
    if (cudaGetDevice(&dev) != cudaSuccess) return 0;
    if (cudaDeviceGetAttribute(&n, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess) return 0;
    return n;
}

namespace {
std::atomic<int> g_sm_budget{0};
}
int sm_budget() { return g_sm_budget.load(std::memory_order_relaxed); }
void set_sm_budget(int sms) { g_sm_budget.store(sms, std::memory_order_relaxed); }
std::atomic<int> g_lm_head_pairing{0};
int lm_head_pairing() { return g_lm_head_pairing.load(std::memory_order_relaxed); }
void set_lm_head_pairing(int on) { g_lm_head_pairing.store(on != 0 ? 1 : 0, std::memory_order_relaxed); }

rpx_status_t check_arch() {
    int dev = 0, major = 0;
    if (cudaGetDevice(&dev) != cudaSuccess) return RPX_ERR_CUDA;
    if (cudaDeviceGetAttribute(&major, cudaDevAttrComputeCapabilityMajor, dev) != cudaSuccess) return RPX_ERR_CUDA;
    return major == 10 ? RPX_OK : RPX_ERR_ARCH;
}

rpx_status_t launch_cast_f32_bf16(const float* src, int64_t src_row_stride, __nv_bfloat16_raw* dst, int64_t rows,
                                  int64_t cols, cudaStream_t stream) {
    const int64_t total = rows * cols;
    if (total == 0) return RPX_OK;
    const int threads = 256;
    int64_t blocks = (total + threads - 1) / threads;
    const int64_t cap = static_cast<int64_t>(sm_count() > 0 ? sm_count() : 148) * 16;
    if (blocks > cap) blocks = cap;
    cast_f32_bf16_kernel<<<static_cast<unsigned>(blocks), threads, 0, stream>>>(
        src, src_row_stride, reinterpret_cast<__nv_bfloat16*>(dst), rows, cols);
    return cudaGetLastError() == cudaSuccess ? RPX_OK : RPX_ERR_CUDA;
}

}  // namespace rpx
