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

int qg_test_gemv_mode(qg_ctx* ctx, int mode) {
    if (!ctx) return QG_ERR_NULL;
    if (mode < 0 || mode > 7 || (mode & 6) == 6) return QG_ERR_SHAPE;
    ctx->gemv_mode = mode;
    return QG_OK;
}

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

// The cache is a table of TMAP_CACHE entries in sets of TMAP_WAYS: a key hashes to one set, a miss replaces the set's
// ways in turn.  A hit or a fresh encode is copied out, so nothing a caller holds changes when a later lookup replaces
// the entry.
static int tmap_lookup(qg_ctx* ctx, CUtensorMap* out, const TmapEntry& key, uint32_t rank) {
    uint64_t h = reinterpret_cast<uintptr_t>(key.base) >> 4;
    h ^= key.inner * 0x9E3779B97F4A7C15ull;
    h ^= (static_cast<uint64_t>(key.box_inner) << 40) ^ (static_cast<uint64_t>(key.box_rows) << 24) ^ (key.rows << 3) ^
         static_cast<uint64_t>(key.swz) ^ (key.planes << 51);
    h *= 0xD6E8FEB86659FD93ull;
    const int set = static_cast<int>((h >> 32) % (TMAP_CACHE / TMAP_WAYS)) * TMAP_WAYS;
    for (int w = 0; w < TMAP_WAYS; ++w) {
        const TmapEntry& e = ctx->tmaps[set + w];
        if (e.base == key.base && e.inner == key.inner && e.rows == key.rows && e.box_inner == key.box_inner &&
            e.box_rows == key.box_rows && e.row_stride == key.row_stride && e.planes == key.planes &&
            e.plane_stride == key.plane_stride && e.box_planes == key.box_planes && e.dt == key.dt &&
            e.elem_bytes == key.elem_bytes && e.swz == key.swz) {
            *out = e.map;
            return QG_OK;
        }
    }
    int way = -1;
    for (int w = 0; w < TMAP_WAYS && way < 0; ++w)
        if (!ctx->tmaps[set + w].base) way = w;
    if (way < 0) way = static_cast<int>(ctx->tmap_next++ % TMAP_WAYS);
    TmapEntry& e = ctx->tmaps[set + way];
    cuuint64_t dims[3] = {key.inner, key.rows, key.planes};
    cuuint64_t strides[2] = {key.row_stride, key.plane_stride};
    cuuint32_t box[3] = {key.box_inner, key.box_rows, key.box_planes};
    cuuint32_t estr[3] = {1, 1, 1};
    e.base = nullptr;      // not a valid entry while it is being rewritten
    const CUresult r = ctx->encode_tiled(&e.map, static_cast<CUtensorMapDataType>(key.dt), rank, const_cast<void*>(key.base),
                                         dims, strides, box, estr, CU_TENSOR_MAP_INTERLEAVE_NONE,
                                         static_cast<CUtensorMapSwizzle>(key.swz), CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                                         CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
    if (r != CUDA_SUCCESS) return QG_ERR_CUDA;
    const CUtensorMap keep = e.map;
    e = key;
    e.map = keep;
    *out = e.map;
    return QG_OK;
}

int get_tmap_2d(qg_ctx* ctx, CUtensorMap* out, CUtensorMapDataType dt, int elem_bytes, const void* base,
                uint64_t inner, uint64_t rows, uint32_t box_inner, uint32_t box_rows, CUtensorMapSwizzle swz,
                uint64_t row_stride_bytes) {
    TmapEntry key{};
    key.base = base; key.inner = inner; key.rows = rows;
    key.row_stride = row_stride_bytes ? row_stride_bytes : inner * static_cast<uint64_t>(elem_bytes);
    key.box_inner = box_inner; key.box_rows = box_rows;
    key.planes = 0; key.plane_stride = 0; key.box_planes = 0;
    key.dt = static_cast<int>(dt); key.elem_bytes = elem_bytes; key.swz = static_cast<int>(swz);
    return tmap_lookup(ctx, out, key, 2);
}

int get_tmap_3d(qg_ctx* ctx, CUtensorMap* out, CUtensorMapDataType dt, int elem_bytes, const void* base,
                uint64_t inner, uint64_t rows, uint64_t planes, uint64_t plane_stride_bytes, uint32_t box_inner,
                uint32_t box_rows, uint32_t box_planes, CUtensorMapSwizzle swz) {
    TmapEntry key{};
    key.base = base; key.inner = inner; key.rows = rows; key.row_stride = inner * static_cast<uint64_t>(elem_bytes);
    key.box_inner = box_inner; key.box_rows = box_rows;
    key.planes = planes; key.plane_stride = plane_stride_bytes; key.box_planes = box_planes;
    key.dt = static_cast<int>(dt); key.elem_bytes = elem_bytes; key.swz = static_cast<int>(swz);
    return tmap_lookup(ctx, out, key, 3);
}
}  // namespace qg
