// Host-side state shared by the tensor-core kernels: the driver's tensor-map encoder and a cache
// of the weight matrices' tensor maps.  Internal to the library.
#pragma once
#include <cuda.h>

#include <map>
#include <utility>

#include "gemm_tc.h"

namespace beagle {

typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*, const cuuint64_t*,
                                  const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave, CUtensorMapSwizzle,
                                  CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

struct TcPlan {
    EncodeTiledFn encode = nullptr;
    beagle_config cfg;
    beagle_weights w;
    std::map<std::pair<const void*, int>, CUtensorMap> weight_maps;   // (pointer, box rows) -> map
    struct Packed { const void* tiles; int N, K, elt_bytes; CUtensorMap map; };
    std::map<const void*, Packed> packed;                             // row-major weight pointer -> its tile-major copy
    int sm_count = 148;
    CUtensorMap cache_k, cache_v;      // the K/V cache as [rows, head_dim] for the staged decode attention
    bool cache_maps_ok = false;
};

// K-major bf16 matrix [rows, K] (row stride ld elements), box = 64 columns x box_rows rows,
// 128-byte swizzle, out-of-range elements read as zero.
bool tc_encode_map(TcPlan* p, CUtensorMap* out, const void* base, long long rows, long long K, long long ld, int box_rows);
// An MN-major bf16 operand: stored [krows, feat] row-major (row stride ld elements); box = 64 features x 64 k-rows.
bool tc_encode_map_mn(TcPlan* p, CUtensorMap* out, const void* base, long long feat, long long krows, long long ld);
// The same for a K-major matrix of bytes (FP8): box = 128 columns x box_rows rows.
bool tc_encode_map_u8(TcPlan* p, CUtensorMap* out, const void* base, long long rows, long long K, long long ld, int box_rows);
const CUtensorMap* tc_weight_map_u8(TcPlan* p, const void* W, int rows, int K, int box_rows);
// Cached map of a weight matrix [rows, K] (dense, ld = K).
const CUtensorMap* tc_weight_map(TcPlan* p, const void* W, int rows, int K, int box_rows);

}  // namespace beagle
