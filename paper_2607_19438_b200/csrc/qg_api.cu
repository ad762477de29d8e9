// Context management, error strings and tensor-map encoding for the quantised GEMM library.
#include <new>

#include "qg_internal.h"

extern "C" {

const char* qg_strerror(int code) {
    switch (code) {
        case QG_OK: return "ok";
        case QG_ERR_NULL: return "a required pointer is NULL";
        case QG_ERR_SHAPE: return "shape not accepted (K % 256, N % 8, H % 8, 1 <= k <= E <= 1024, F % 64)";
        case QG_ERR_ALIGN: return "pointer not 16-byte aligned";
        case QG_ERR_WORKSPACE: return "workspace missing or too small";
        case QG_ERR_ARCH: return "device is not compute capability 10.x (sm_100a kernels only)";
        case QG_ERR_CUDA: return "CUDA runtime or driver call failed";
        case QG_ERR_TIMEOUT: return "a bounded device-side wait expired";
        case QG_ERR_TOO_LARGE: return "problem exceeds the built-in scratch of moe_route_static (ceil(M/32)*E <= 65536)";
        default: return "unknown error code";
    }
}

int qg_create(qg_ctx** out, int device) {
    if (!out) return QG_ERR_NULL;
    *out = nullptr;
    cudaDeviceProp prop;
    if (cudaGetDeviceProperties(&prop, device) != cudaSuccess) { cudaGetLastError(); return QG_ERR_CUDA; }
    if (prop.major != 10) return QG_ERR_ARCH;
    if (cudaSetDevice(device) != cudaSuccess) { cudaGetLastError(); return QG_ERR_CUDA; }
    qg_ctx* ctx = new (std::nothrow) qg_ctx();
    if (!ctx) return QG_ERR_CUDA;
    ctx->device = device;
    ctx->sm_count = prop.multiProcessorCount;
    void* fn = nullptr;
    cudaDriverEntryPointQueryResult qres;
    if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &fn, cudaEnableDefault, &qres) != cudaSuccess || !fn ||
        qres != cudaDriverEntryPointSuccess) {
        cudaGetLastError();
        delete ctx;
        return QG_ERR_CUDA;
    }
    ctx->encode_tiled = reinterpret_cast<decltype(ctx->encode_tiled)>(fn);
    if (cudaMalloc(&ctx->d_status, sizeof(int)) != cudaSuccess || cudaMemset(ctx->d_status, 0, sizeof(int)) != cudaSuccess) {
        cudaGetLastError();
        delete ctx;
        return QG_ERR_CUDA;
    }
    *out = ctx;
    return QG_OK;
}

int qg_destroy(qg_ctx* ctx) {
    if (!ctx) return QG_ERR_NULL;
    cudaFree(ctx->d_status);
    delete ctx;
    return QG_OK;
}

int qg_poll_status(qg_ctx* ctx, void* stream) {
    if (!ctx) return QG_ERR_NULL;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    int host = 0;
    if (cudaStreamSynchronize(st) != cudaSuccess) { cudaGetLastError(); return QG_ERR_CUDA; }
    if (cudaMemcpy(&host, ctx->d_status, sizeof(int), cudaMemcpyDeviceToHost) != cudaSuccess) { cudaGetLastError(); return QG_ERR_CUDA; }
    if (host != 0) cudaMemset(ctx->d_status, 0, sizeof(int));
    return host;
}

}  // extern "C"

namespace qg {
int make_tmap_2d(qg_ctx* ctx, CUtensorMap* out, CUtensorMapDataType dt, int elem_bytes, const void* base,
                 uint64_t inner, uint64_t rows, uint32_t box_inner, uint32_t box_rows, CUtensorMapSwizzle swz) {
    cuuint64_t dims[2] = {inner, rows};
    cuuint64_t strides[1] = {inner * static_cast<uint64_t>(elem_bytes)};
    cuuint32_t box[2] = {box_inner, box_rows};
    cuuint32_t estr[2] = {1, 1};
    CUresult r = ctx->encode_tiled(out, dt, 2, const_cast<void*>(base), dims, strides, box, estr,
                                   CU_TENSOR_MAP_INTERLEAVE_NONE, swz, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                                   CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
    return r == CUDA_SUCCESS ? QG_OK : QG_ERR_CUDA;
}
}  // namespace qg
