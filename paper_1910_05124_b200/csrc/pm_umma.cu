// bf16 grouped GEMMs.  Scaffold: routes to the SIMT kernels until the tcgen05 path lands.
#include "pm_umma.cuh"

namespace pm {
struct UmmaPlan { int dummy; };
pm_status umma_plan_create(UmmaPlan** out, const TickArgs&, const std::vector<StageDev>&, std::string&) {
  *out = new UmmaPlan{0};
  return PM_OK;
}
void umma_plan_destroy(UmmaPlan* plan) { delete plan; }
cudaError_t umma_launch(UmmaPlan*, const TickArgs& t, int mode, int lvl, cudaStream_t stream) {
  return launch_simt_gemm(t, PM_BF16, mode, lvl, stream);
}
}  // namespace pm
