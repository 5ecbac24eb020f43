// bf16 tensor-core grouped GEMMs of the pipeline (tcgen05 + TMEM + TMA): interface to the host code.
#pragma once
#include <string>
#include <vector>
#include "pm_tick.cuh"

namespace pm {

struct UmmaPlan;   // tensor maps and launch geometry, built once per context

pm_status umma_plan_create(UmmaPlan** out, const TickArgs& t, const std::vector<StageDev>& st, std::string& err);
void umma_plan_destroy(UmmaPlan* plan);
// mode: 0 forward, 1 dgrad (corrected weights formed in the operand-load path), 2 wgrad.
cudaError_t umma_launch(UmmaPlan* plan, const TickArgs& t, int mode, int lvl, cudaStream_t stream);

}  // namespace pm
