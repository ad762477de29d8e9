// Internal declarations shared by the translation units of the library (not part of the ABI).
#pragma once
#include <cuda.h>
#include <cuda_runtime.h>
#include <stdint.h>

#include <utility>

#include "../../include/qgemm.h"

namespace qg {
// One cached tensor map: the key is everything cuTensorMapEncodeTiled was given.
struct TmapEntry {
    const void* base;
    uint64_t inner, rows, row_stride;
    uint32_t box_inner, box_rows;
    uint64_t planes, plane_stride;   // third dimension of a 3-D map (0 for 2-D maps)
    uint32_t box_planes;
    int dt, elem_bytes, swz;
    CUtensorMap map;
};
constexpr int TMAP_CACHE = 2048, TMAP_WAYS = 8;   // entries, entries per hashed set
constexpr uint32_t DEFAULT_WAIT_LIMIT = 1u << 18;   // polls; an unsatisfied try_wait poll lasts about 4 us: about a second
// Slots of qg_ctx::attr_set, one per kernel instantiation that needs the dynamic shared-memory attribute.
enum AttrSlot {
    ATTR_GEMM = 0,          // 18 slots: format (2) x token tile (3) x epilogue (3)
    ATTR_GEMV = 18,         // 2: Q8, Q4
    ATTR_ATTN = 20,         // 3: head dimensions
    ATTR_ROUTER_1 = 23,
    ATTR_GEMM_SK = 24,      // 6: format (2) x token tile (3), stream-K
    ATTR_MX_192 = 30,
    ATTR_ROUTER_4 = 31,
    ATTR_MX_MOE = 32,       // 2: down, gate/up
    ATTR_MX_256 = 34,
    ATTR_GEMV_RING = 35,    // 4: format (2) x more than eight tokens (2)
    ATTR_SLOTS = 39
};
}  // namespace qg

struct qg_ctx {
    int device;
    int sm_count;
    int* d_status;  // device status word: 0, or the first QG_ERR_* a kernel recorded
    CUresult (*encode_tiled)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*,
                             const cuuint64_t*, const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave,
                             CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);
    int force_bt;              // QG_FORCE_BT at creation (0: heuristic)
    uint32_t wait_limit;       // polls per bounded device wait
    int skip_kb;               // test hook, consumed by the next GEMM launch (-1: none)
    bool attr_set[qg::ATTR_SLOTS];        // per kernel instantiation: dynamic shared-memory attribute set on this device
    qg::TmapEntry tmaps[qg::TMAP_CACHE];   // tensor maps of recent calls (weights and buffers recur every layer)
    unsigned tmap_next;        // replacement counter
    bool pdl;                  // launch kernels with programmatic stream serialization (QG_NO_PDL=1 turns it off)
    float* sk_partial;         // stream-K: one fp32 partial tile (256 tokens x 128 rows) per CTA
    int* sk_flags;             // stream-K: two counters per CTA, zero between launches
    int streamk_mode;          // QG_STREAMK at creation: -1 heuristic (default), 0 never, 1 whenever legal
    float* gemv_partial;       // K-slice partial sums of qgemm_small_m, [slices][16][N] fp32
    size_t gemv_partial_bytes;
    int* gemv_tickets;         // one arrival counter per 64-row tile, zero between launches
    int gemv_ticket_count;
    int gemv_mode;             // test hook (qg_test_gemv_mode): bit 0 no clusters, bit 1 always the ring kernel, bit 2 never
    int gemv_max_clusters[4][9];   // ring kernel, per instantiation and cluster size: clusters that fit at once (0 unknown, -1 none)
    long long* stats;          // profiling builds only
};

namespace qg {
// Launches `kern`; with ctx->pdl the launch carries the programmatic-serialization attribute, so the kernel's prologue
// may overlap the tail of the kernel before it in the stream (every kernel of this library calls pdl_wait() before it
// reads or writes anything an earlier kernel may touch).
template <typename... KArgs, typename... Args>
inline cudaError_t launch_kernel(const qg_ctx* ctx, void (*kern)(KArgs...), dim3 grid, dim3 block, size_t smem,
                                 cudaStream_t st, Args&&... args) {
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = grid; cfg.blockDim = block; cfg.dynamicSmemBytes = smem; cfg.stream = st;
    cudaLaunchAttribute at[1];
    at[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    at[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = at;
    cfg.numAttrs = ctx->pdl ? 1 : 0;
    return cudaLaunchKernelEx(&cfg, kern, std::forward<Args>(args)...);
}
inline bool aligned16(const void* p) { return (reinterpret_cast<uintptr_t>(p) & 15) == 0; }
// QG_OK if the calling thread's current device is the context's, else QG_ERR_DEVICE.
int check_device(const qg_ctx* ctx);
// A 2-D row-major tensor map (inner = contiguous extent in elements, box in elements, row_stride_bytes = distance
// between rows, 0 = packed): looked up in the context's cache, encoded on a miss, and copied to *out (the caller's own
// copy: a later lookup may replace the cached entry).
int get_tmap_2d(qg_ctx* ctx, CUtensorMap* out, CUtensorMapDataType dt, int elem_bytes, const void* base,
                uint64_t inner, uint64_t rows, uint32_t box_inner, uint32_t box_rows, CUtensorMapSwizzle swz,
                uint64_t row_stride_bytes = 0);
// The same with a third dimension: `planes` planes of `rows` rows, plane_stride_bytes apart; box = box_inner x box_rows x
// box_planes, which lands in shared memory plane after plane.
int get_tmap_3d(qg_ctx* ctx, CUtensorMap* out, CUtensorMapDataType dt, int elem_bytes, const void* base,
                uint64_t inner, uint64_t rows, uint64_t planes, uint64_t plane_stride_bytes, uint32_t box_inner,
                uint32_t box_rows, uint32_t box_planes, CUtensorMapSwizzle swz);
}  // namespace qg
