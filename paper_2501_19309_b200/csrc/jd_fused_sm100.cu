// placeholder until the tensor-core kernel lands
#include "jd_kernels.h"
namespace jd {
bool fused_supported(int, int, int, int, int, FusedPlan*) { return false; }
int run_fused(const CallParams&, const Workspace&, const CUtensorMap&, const CUtensorMap&, const void*, const void*,
              const FusedPlan&, cudaStream_t, cudaError_t* err) { *err = cudaErrorNotSupported; return -1; }
}
