// Context management, error strings and tensor-map encoding for the quantised GEMM library.
#include <new>
#include <stdlib.h>

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
        case QG_ERR_DEVICE: return "the current CUDA device is not the context's device";
        default: return "unknown error code";
    }
}

int qg_create(qg_ctx** out, int device) {
    if (!out) return QG_ERR_NULL;
    *out = nullptr;
    cudaDeviceProp prop;
    if (cudaGetDeviceProperties(&prop, device) != cudaSuccess) { cudaGetLastError(); return QG_ERR_CUDA; }
    if (prop.major != 10) return QG_ERR_ARCH;
    int prev = -1;
    if (cudaGetDevice(&prev) != cudaSuccess) { cudaGetLastError(); return QG_ERR_CUDA; }
    if (cudaSetDevice(device) != cudaSuccess) { cudaGetLastError(); return QG_ERR_CUDA; }
    struct Restore {       // the caller's current device is left as it was
        int dev;
        ~Restore() { if (dev >= 0) cudaSetDevice(dev); }
    } restore{prev};
    qg_ctx* ctx = new (std::nothrow) qg_ctx();
    if (!ctx) return QG_ERR_CUDA;
    ctx->device = device;
    ctx->sm_count = prop.multiProcessorCount;
    ctx->wait_limit = qg::DEFAULT_WAIT_LIMIT;
    ctx->skip_kb = -1;
    const char* no_pdl = getenv("QG_NO_PDL");
    ctx->pdl = !(no_pdl && no_pdl[0] == '1');
    if (const char* f = getenv("QG_FORCE_BT")) {   // tile-shape override for sweeps, read once
        const int v = atoi(f);
        if (v == 128 || v == 192 || v == 256) ctx->force_bt = v;
    }
    void* fn = nullptr;
    cudaDriverEntryPointQueryResult qres;
    if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &fn, cudaEnableDefault, &qres) != cudaSuccess || !fn ||
        qres != cudaDriverEntryPointSuccess) {
        cudaGetLastError();
        delete ctx;
        return QG_ERR_CUDA;
    }
    ctx->encode_tiled = reinterpret_cast<decltype(ctx->encode_tiled)>(fn);
    ctx->streamk_mode = -1;
    if (const char* f = getenv("QG_STREAMK")) ctx->streamk_mode = (f[0] == '0') ? 0 : (f[0] == '1') ? 1 : -1;
    ctx->gemv_partial_bytes = static_cast<size_t>(32) << 20;
    ctx->gemv_ticket_count = 4096;
    if (cudaMalloc(&ctx->d_status, sizeof(int)) != cudaSuccess || cudaMemset(ctx->d_status, 0, sizeof(int)) != cudaSuccess ||
        cudaMalloc(&ctx->sk_partial, static_cast<size_t>(ctx->sm_count) * 256 * 128 * sizeof(float)) != cudaSuccess ||
        cudaMalloc(&ctx->sk_flags, sizeof(int) * 2 * ctx->sm_count) != cudaSuccess ||
        cudaMemset(ctx->sk_flags, 0, sizeof(int) * 2 * ctx->sm_count) != cudaSuccess ||
        cudaMalloc(&ctx->gemv_partial, ctx->gemv_partial_bytes) != cudaSuccess ||
        cudaMalloc(&ctx->gemv_tickets, sizeof(int) * ctx->gemv_ticket_count) != cudaSuccess ||
        cudaMemset(ctx->gemv_tickets, 0, sizeof(int) * ctx->gemv_ticket_count) != cudaSuccess) {
        cudaGetLastError();
        cudaFree(ctx->d_status); cudaFree(ctx->gemv_partial); cudaFree(ctx->gemv_tickets);
        cudaFree(ctx->sk_partial); cudaFree(ctx->sk_flags);
        delete ctx;
        return QG_ERR_CUDA;
    }
    *out = ctx;
    return QG_OK;
}

int qg_destroy(qg_ctx* ctx) {
    if (!ctx) return QG_ERR_NULL;
    cudaFree(ctx->d_status);
    cudaFree(ctx->gemv_partial);
    cudaFree(ctx->gemv_tickets);
    cudaFree(ctx->sk_partial);
    cudaFree(ctx->sk_flags);
    delete ctx;
    return QG_OK;
}

int qg_poll_status(qg_ctx* ctx, void* stream) {
    if (!ctx) return QG_ERR_NULL;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    int host = 0;
    if (cudaStreamSynchronize(st) != cudaSuccess) { cudaGetLastError(); return QG_ERR_CUDA; }
    if (cudaMemcpy(&host, ctx->d_status, sizeof(int), cudaMemcpyDeviceToHost) != cudaSuccess) { cudaGetLastError(); return QG_ERR_CUDA; }
    if (host != 0) {
        // a kernel gave up: clear the status word and the cross-CTA counters it may have left half-way, so that the
        // next launch starts clean
        cudaMemset(ctx->d_status, 0, sizeof(int));
        cudaMemset(ctx->sk_flags, 0, sizeof(int) * 2 * ctx->sm_count);
        cudaMemset(ctx->gemv_tickets, 0, sizeof(int) * ctx->gemv_ticket_count);
    }
    return host;
}

int qg_set_schedule(qg_ctx* ctx, int token_tile, int streamk_mode) {
    if (!ctx) return QG_ERR_NULL;
    if (token_tile != 0 && token_tile != 128 && token_tile != 192 && token_tile != 256) return QG_ERR_SHAPE;
    if (streamk_mode < -1 || streamk_mode > 1) return QG_ERR_SHAPE;
    ctx->force_bt = token_tile;
    ctx->streamk_mode = streamk_mode;
    return QG_OK;
}

#ifdef QG_PROFILE
// profiling builds only: device buffer for the GEMM kernel's cycle counters and milestones
void qg_debug_set_stats(qg_ctx* ctx, long long* dev_buf) { if (ctx) ctx->stats = dev_buf; }
#endif

int qg_test_inject(qg_ctx* ctx, unsigned wait_limit_polls, int skip_kblock) {
    if (!ctx) return QG_ERR_NULL;
    ctx->wait_limit = wait_limit_polls ? wait_limit_polls : qg::DEFAULT_WAIT_LIMIT;
    ctx->skip_kb = skip_kblock;
    return QG_OK;
}

}  // extern "C"

namespace qg {
int check_device(const qg_ctx* ctx) {
    int dev = -1;
    if (cudaGetDevice(&dev) != cudaSuccess) { cudaGetLastError(); return QG_ERR_CUDA; }
    return dev == ctx->device ? QG_OK : QG_ERR_DEVICE;
}

int get_tmap_2d(qg_ctx* ctx, const CUtensorMap** out, CUtensorMapDataType dt, int elem_bytes, const void* base,
                uint64_t inner, uint64_t rows, uint32_t box_inner, uint32_t box_rows, CUtensorMapSwizzle swz,
                uint64_t row_stride_bytes) {
    if (row_stride_bytes == 0) row_stride_bytes = inner * static_cast<uint64_t>(elem_bytes);
    for (int i = 0; i < ctx->tmap_count; ++i) {
        const TmapEntry& e = ctx->tmaps[i];
        if (e.base == base && e.inner == inner && e.rows == rows && e.box_inner == box_inner && e.box_rows == box_rows &&
            e.row_stride == row_stride_bytes && e.planes == 0 &&
            e.dt == static_cast<int>(dt) && e.elem_bytes == elem_bytes && e.swz == static_cast<int>(swz)) {
            *out = &e.map;
            return QG_OK;
        }
    }
    TmapEntry& e = ctx->tmaps[ctx->tmap_next];
    cuuint64_t dims[2] = {inner, rows};
    cuuint64_t strides[1] = {row_stride_bytes};
    cuuint32_t box[2] = {box_inner, box_rows};
    cuuint32_t estr[2] = {1, 1};
    e.base = nullptr;      // not a valid entry while it is being rewritten
    CUresult r = ctx->encode_tiled(&e.map, dt, 2, const_cast<void*>(base), dims, strides, box, estr,
                                   CU_TENSOR_MAP_INTERLEAVE_NONE, swz, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                                   CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
    if (r != CUDA_SUCCESS) return QG_ERR_CUDA;
    e.base = base; e.inner = inner; e.rows = rows; e.row_stride = row_stride_bytes; e.box_inner = box_inner; e.box_rows = box_rows;
    e.planes = 0; e.plane_stride = 0; e.box_planes = 0;
    e.dt = static_cast<int>(dt); e.elem_bytes = elem_bytes; e.swz = static_cast<int>(swz);
    *out = &e.map;
    ctx->tmap_next = (ctx->tmap_next + 1) % TMAP_CACHE;
    if (ctx->tmap_count < TMAP_CACHE) ++ctx->tmap_count;
    return QG_OK;
}

int get_tmap_3d(qg_ctx* ctx, const CUtensorMap** out, CUtensorMapDataType dt, int elem_bytes, const void* base,
                uint64_t inner, uint64_t rows, uint64_t planes, uint64_t plane_stride_bytes, uint32_t box_inner,
                uint32_t box_rows, uint32_t box_planes, CUtensorMapSwizzle swz) {
    const uint64_t row_stride_bytes = inner * static_cast<uint64_t>(elem_bytes);
    for (int i = 0; i < ctx->tmap_count; ++i) {
        const TmapEntry& e = ctx->tmaps[i];
        if (e.base == base && e.inner == inner && e.rows == rows && e.box_inner == box_inner && e.box_rows == box_rows &&
            e.row_stride == row_stride_bytes && e.planes == planes && e.plane_stride == plane_stride_bytes &&
            e.box_planes == box_planes &&
            e.dt == static_cast<int>(dt) && e.elem_bytes == elem_bytes && e.swz == static_cast<int>(swz)) {
            *out = &e.map;
            return QG_OK;
        }
    }
    TmapEntry& e = ctx->tmaps[ctx->tmap_next];
    cuuint64_t dims[3] = {inner, rows, planes};
    cuuint64_t strides[2] = {row_stride_bytes, plane_stride_bytes};
    cuuint32_t box[3] = {box_inner, box_rows, box_planes};
    cuuint32_t estr[3] = {1, 1, 1};
    e.base = nullptr;      // not a valid entry while it is being rewritten
    CUresult r = ctx->encode_tiled(&e.map, dt, 3, const_cast<void*>(base), dims, strides, box, estr,
                                   CU_TENSOR_MAP_INTERLEAVE_NONE, swz, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                                   CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
    if (r != CUDA_SUCCESS) return QG_ERR_CUDA;
    e.base = base; e.inner = inner; e.rows = rows; e.row_stride = row_stride_bytes; e.box_inner = box_inner; e.box_rows = box_rows;
    e.planes = planes; e.plane_stride = plane_stride_bytes; e.box_planes = box_planes;
    e.dt = static_cast<int>(dt); e.elem_bytes = elem_bytes; e.swz = static_cast<int>(swz);
    *out = &e.map;
    ctx->tmap_next = (ctx->tmap_next + 1) % TMAP_CACHE;
    if (ctx->tmap_count < TMAP_CACHE) ++ctx->tmap_count;
    return QG_OK;
}
}  // namespace qg
