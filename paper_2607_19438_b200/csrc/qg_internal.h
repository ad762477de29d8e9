// Internal declarations shared by the translation units of the library (not part of the ABI).
#pragma once
#include <cuda.h>
#include <cuda_runtime.h>
#include <stdint.h>

#include "../../include/qgemm.h"

struct qg_ctx {
    int device;
    int sm_count;
    int* d_status;  // device status word: 0, or the first QG_ERR_* a kernel recorded
    CUresult (*encode_tiled)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*,
                             const cuuint64_t*, const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave,
                             CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);
};

namespace qg {
inline bool aligned16(const void* p) { return (reinterpret_cast<uintptr_t>(p) & 15) == 0; }
// Encodes a 2-D row-major tensor map; inner = contiguous extent in elements, box in elements.
int make_tmap_2d(qg_ctx* ctx, CUtensorMap* out, CUtensorMapDataType dt, int elem_bytes, const void* base,
                 uint64_t inner, uint64_t rows, uint32_t box_inner, uint32_t box_rows, CUtensorMapSwizzle swz);
}  // namespace qg
