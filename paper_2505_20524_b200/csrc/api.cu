// Host-side state shared by every entry point: error text, the device status word, architecture check,
// and the tensor-map encoder fetched from the driver at run time (the library does not link libcuda).
#include <stdarg.h>
#include <stdio.h>

#include "common.cuh"

namespace fp8dpa {

static thread_local char g_err[512] = "no error";

void set_error(const char *fmt, ...)
{
    va_list ap;
    va_start(ap, fmt);
    vsnprintf(g_err, sizeof(g_err), fmt, ap);
    va_end(ap);
}

// One status word per device (each device that loads the module gets its own copy of the symbol).
__device__ int g_device_status = 0;

static const int kMaxDevices = 64;
static int *g_status_ptr[kMaxDevices] = {nullptr};
static int g_arch_ok[kMaxDevices] = {0};   // 0 unknown, 1 ok, -1 wrong arch
static int g_sm_count[kMaxDevices] = {0};

static int current_device()
{
    int dev = -1;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= kMaxDevices) return -1;
    return dev;
}

int *device_status_ptr()
{
    int dev = current_device();
    if (dev < 0) return nullptr;
    if (!g_status_ptr[dev]) {
        void *p = nullptr;
        if (cudaGetSymbolAddress(&p, g_device_status) != cudaSuccess) {
            set_error("cudaGetSymbolAddress(status word) failed: %s", cudaGetErrorString(cudaGetLastError()));
            return nullptr;
        }
        g_status_ptr[dev] = static_cast<int *>(p);
    }
    return g_status_ptr[dev];
}

int check_arch()
{
    int dev = current_device();
    if (dev < 0) {
        set_error("no current CUDA device: %s", cudaGetErrorString(cudaGetLastError()));
        return FP8_ERR_CUDA;
    }
    if (g_arch_ok[dev] == 0) {
        int major = 0, sms = 0;
        if (cudaDeviceGetAttribute(&major, cudaDevAttrComputeCapabilityMajor, dev) != cudaSuccess ||
            cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess) {
            set_error("cudaDeviceGetAttribute failed: %s", cudaGetErrorString(cudaGetLastError()));
            return FP8_ERR_CUDA;
        }
        g_arch_ok[dev] = (major == 10) ? 1 : -1;
        g_sm_count[dev] = sms;
    }
    if (g_arch_ok[dev] < 0) {
        set_error("this library only runs on compute capability 10.x (sm_100a); no fallback exists");
        return FP8_ERR_ARCH;
    }
    return FP8_OK;
}

int sm_count()
{
    int dev = current_device();
    return (dev >= 0 && g_sm_count[dev] > 0) ? g_sm_count[dev] : 148;
}

typedef CUresult (*encode_tiled_fn)(CUtensorMap *, CUtensorMapDataType, cuuint32_t, void *, const cuuint64_t *,
                                    const cuuint64_t *, const cuuint32_t *, const cuuint32_t *,
                                    CUtensorMapInterleave, CUtensorMapSwizzle, CUtensorMapL2promotion,
                                    CUtensorMapFloatOOBfill);
static encode_tiled_fn g_encode = nullptr;

static int load_encoder()
{
    if (g_encode) return FP8_OK;
    void *fn = nullptr;
    cudaDriverEntryPointQueryResult q;
    cudaError_t e = cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &fn, cudaEnableDefault, &q);
    if (e != cudaSuccess || q != cudaDriverEntryPointSuccess || !fn) {
        set_error("cuTensorMapEncodeTiled not available from the driver (%s)", cudaGetErrorString(e));
        return FP8_ERR_CUDA;
    }
    g_encode = reinterpret_cast<encode_tiled_fn>(fn);
    return FP8_OK;
}

int make_tmap_2d_u8(CUtensorMap *map, const void *base, uint64_t rows, uint64_t cols, uint64_t pitch,
                    uint32_t box_rows, uint32_t box_cols)
{
    int rc = load_encoder();
    if (rc != FP8_OK) return rc;
    cuuint64_t dims[2] = {cols, rows};
    cuuint64_t strides[1] = {pitch};
    cuuint32_t box[2] = {box_cols, box_rows};
    cuuint32_t estr[2] = {1, 1};
    CUresult r = g_encode(map, CU_TENSOR_MAP_DATA_TYPE_UINT8, 2, const_cast<void *>(base), dims, strides, box, estr,
                          CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B,
                          CU_TENSOR_MAP_L2_PROMOTION_L2_256B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
    if (r != CUDA_SUCCESS) {
        set_error("cuTensorMapEncodeTiled failed (CUresult %d) rows=%llu cols=%llu pitch=%llu box=%ux%u", (int)r,
                  (unsigned long long)rows, (unsigned long long)cols, (unsigned long long)pitch, box_rows, box_cols);
        return FP8_ERR_CUDA;
    }
    return FP8_OK;
}

// Rank-3 map over a [B, N, H*d] byte tensor: box = [1, box_rows, box_cols]; swizzle 128 B when box_cols is
// 128, 64 B when it is 64.
int make_tmap_3d_u8(CUtensorMap *map, const void *base, uint64_t d0_cols, uint64_t d1_rows, uint64_t d2_batch,
                    uint32_t box_cols, uint32_t box_rows)
{
    int rc = load_encoder();
    if (rc != FP8_OK) return rc;
    cuuint64_t dims[3] = {d0_cols, d1_rows, d2_batch};
    cuuint64_t strides[2] = {d0_cols, d0_cols * d1_rows};
    cuuint32_t box[3] = {box_cols, box_rows, 1};
    cuuint32_t estr[3] = {1, 1, 1};
    CUtensorMapSwizzle sw = box_cols == 128 ? CU_TENSOR_MAP_SWIZZLE_128B
                          : box_cols == 64  ? CU_TENSOR_MAP_SWIZZLE_64B
                                            : CU_TENSOR_MAP_SWIZZLE_NONE;
    CUresult r = g_encode(map, CU_TENSOR_MAP_DATA_TYPE_UINT8, 3, const_cast<void *>(base), dims, strides, box, estr,
                          CU_TENSOR_MAP_INTERLEAVE_NONE, sw, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                          CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
    if (r != CUDA_SUCCESS) {
        set_error("cuTensorMapEncodeTiled (rank 3) failed (CUresult %d) dims=%llu,%llu,%llu box=%u,%u", (int)r,
                  (unsigned long long)d0_cols, (unsigned long long)d1_rows, (unsigned long long)d2_batch, box_cols,
                  box_rows);
        return FP8_ERR_CUDA;
    }
    return FP8_OK;
}

// Rank-3 map over a [B, N, C] binary32 tensor without swizzle (used for bulk reduce-add of FP32 tiles).
int make_tmap_3d_f32(CUtensorMap *map, const void *base, uint64_t d0_cols, uint64_t d1_rows, uint64_t d2_batch,
                     uint32_t box_cols, uint32_t box_rows)
{
    int rc = load_encoder();
    if (rc != FP8_OK) return rc;
    cuuint64_t dims[3] = {d0_cols, d1_rows, d2_batch};
    cuuint64_t strides[2] = {d0_cols * 4, d0_cols * d1_rows * 4};
    cuuint32_t box[3] = {box_cols, box_rows, 1};
    cuuint32_t estr[3] = {1, 1, 1};
    CUresult r = g_encode(map, CU_TENSOR_MAP_DATA_TYPE_FLOAT32, 3, const_cast<void *>(base), dims, strides, box, estr,
                          CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_NONE,
                          CU_TENSOR_MAP_L2_PROMOTION_L2_256B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
    if (r != CUDA_SUCCESS) {
        set_error("cuTensorMapEncodeTiled (rank 3, f32) failed (CUresult %d) dims=%llu,%llu,%llu box=%u,%u", (int)r,
                  (unsigned long long)d0_cols, (unsigned long long)d1_rows, (unsigned long long)d2_batch, box_cols,
                  box_rows);
        return FP8_ERR_CUDA;
    }
    return FP8_OK;
}

// Rank-2 map over a [rows, 16] BF16 array (32-byte rows) with the 32-byte swizzle: the right operand of a K = 16
// tcgen05.mma.kind::f16 step, one row per output column.
int make_tmap_2d_bf16x16(CUtensorMap *map, const void *base, uint64_t rows, uint32_t box_rows)
{
    int rc = load_encoder();
    if (rc != FP8_OK) return rc;
    cuuint64_t dims[2] = {16, rows};
    cuuint64_t strides[1] = {32};
    cuuint32_t box[2] = {16, box_rows};
    cuuint32_t estr[2] = {1, 1};
    CUresult r = g_encode(map, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, const_cast<void *>(base), dims, strides, box, estr,
                          CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_32B,
                          CU_TENSOR_MAP_L2_PROMOTION_L2_128B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
    if (r != CUDA_SUCCESS) {
        set_error("cuTensorMapEncodeTiled (rank 2, bf16 x 16) failed (CUresult %d) rows=%llu box=%u", (int)r,
                  (unsigned long long)rows, box_rows);
        return FP8_ERR_CUDA;
    }
    return FP8_OK;
}

// One warp waits on a barrier that nothing ever completes, with a short limit: the path every kernel of the library
// takes when a wait runs out (status word, shared abort flag, orderly return).
__global__ void wait_timeout_selftest_kernel(int *status, long long limit, int *gave_up)
{
    __shared__ __align__(8) uint64_t bar;
    __shared__ int abort_flag;
    const uint32_t b = smem_u32(&bar);
    if (threadIdx.x == 0) {
        mbar_init(b, 1);
        abort_flag = 0;
        mbar_init_fence();
    }
    __syncthreads();
    const WaitCtx ctx{status, &abort_flag, limit};
    const bool got = mbar_wait_warp(b, 0u, ctx);
    if (threadIdx.x == 0) *gave_up = got ? 0 : 1;
}

}  // namespace fp8dpa

extern "C" const char *fp8_last_error(void) { return fp8dpa::g_err; }

extern "C" int fp8_device_status(int *status_out, void *stream)
{
    if (!status_out) {
        fp8dpa::set_error("fp8_device_status: status_out is NULL");
        return FP8_ERR_NULL;
    }
    int *p = fp8dpa::device_status_ptr();
    if (!p) return FP8_ERR_CUDA;
    cudaStream_t s = static_cast<cudaStream_t>(stream);
    FP8_CUDA_CHECK(cudaStreamSynchronize(s));
    FP8_CUDA_CHECK(cudaMemcpy(status_out, p, sizeof(int), cudaMemcpyDeviceToHost));
    FP8_CUDA_CHECK(cudaMemset(p, 0, sizeof(int)));
    return FP8_OK;
}

extern "C" int fp8_selftest_wait_timeout(long long limit_cycles, int *gave_up, void *stream)
{
    if (!gave_up) {
        fp8dpa::set_error("fp8_selftest_wait_timeout: gave_up is NULL");
        return FP8_ERR_NULL;
    }
    if (limit_cycles <= 0 || limit_cycles > (1ll << 31)) {
        fp8dpa::set_error("fp8_selftest_wait_timeout: limit_cycles must be in (0, 2^31], got %lld", limit_cycles);
        return FP8_ERR_SHAPE;
    }
    int rc = fp8dpa::check_arch();
    if (rc != FP8_OK) return rc;
    int *status = fp8dpa::device_status_ptr();
    if (!status) return FP8_ERR_CUDA;
    fp8dpa::wait_timeout_selftest_kernel<<<1, 32, 0, static_cast<cudaStream_t>(stream)>>>(status, limit_cycles, gave_up);
    FP8_CUDA_CHECK(cudaGetLastError());
    return FP8_OK;
}
