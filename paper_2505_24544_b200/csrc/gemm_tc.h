// bf16 tensor-core GEMM (tcgen05 + TMEM + TMA) behind the dense projections.
#pragma once
#include "../../include/beagle.h"
#include "kernels.h"

namespace beagle {

struct TcPlan;   // tensor maps of the weight matrices and launch constants

// Returns nullptr when the tensor-core path cannot serve this configuration.
// *hard_error = 1 when a device is present but the tensor-map encoder could not be obtained.
TcPlan* tc_plan_create(const beagle_config& cfg, const beagle_weights& w, int* hard_error);
void tc_plan_destroy(TcPlan* plan);
// C = A W^T with the fused epilogue `epi` (GemmEpilogue).  Returns the number of kernels launched,
// or -1 when this shape is not covered (the caller then uses the CUDA-core kernel).
int tc_gemm(TcPlan* plan, int epi, const GemmArgs& a, cudaStream_t stream);
// GEMM_ARGMAX_KEYS writes one packed key per (row, 256-column tile): keys [M, tc_argmax_tiles(N)].
int tc_argmax_tiles(int N);
int tc_keys_to_ids(const unsigned long long* keys, int rows, int ntiles, int32_t* ids, cudaStream_t stream);

}  // namespace beagle
