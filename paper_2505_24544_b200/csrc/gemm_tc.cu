#include "gemm_tc.h"

namespace beagle {

struct TcPlan { int unused; };

TcPlan* tc_plan_create(const beagle_config&, const beagle_weights&) { return nullptr; }
void tc_plan_destroy(TcPlan* plan) { delete plan; }
int tc_gemm(TcPlan*, int, const GemmArgs&, cudaStream_t) { return -1; }

}  // namespace beagle
