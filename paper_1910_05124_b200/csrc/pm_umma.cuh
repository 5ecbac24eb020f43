// bf16 tensor-core grouped GEMMs of the pipeline (tcgen05 + TMEM + TMA): interface to the host code.
#pragma once
#include <string>
#include <vector>
#include "pm_tick.cuh"

namespace pm {

struct UmmaPlan;   // tensor maps and launch geometry, built once per context

// Bytes of caller workspace the plan needs (status word + tensor maps).
// dgrad_split_below: see TickArgs::dgrad_split_below (the plan must be created with the same value).
uint64_t umma_workspace_bytes(int T, const std::vector<StageDev>& st, int dgrad_split_below);
// ws_region: device memory of at least umma_workspace_bytes(T, stages), 256-byte aligned.  Synchronises `stream`.
pm_status umma_plan_create(UmmaPlan** out, const TickArgs& t, const std::vector<StageDev>& st, void* ws_region,
                           cudaStream_t stream, std::string& err);
void umma_plan_destroy(UmmaPlan* plan);
// Device word that a CTA sets when one of its bounded waits expired (0 = none).
int* umma_status_word(UmmaPlan* plan);
// Self-test: launches a one-thread kernel whose bounded wait (limit in SM cycles) must expire; it sets the plan's status
// word like a real expiry would and writes 2 to *d_returned.  umma_clear_status resets the status word.
cudaError_t umma_wait_timeout_probe(UmmaPlan* plan, long long limit_cycles, int* d_returned, cudaStream_t stream);
cudaError_t umma_clear_status(UmmaPlan* plan, cudaStream_t stream);
// mode: 0 forward, 1 dgrad (corrected weights formed in the operand-load path), 2 wgrad.
cudaError_t umma_launch(UmmaPlan* plan, const TickArgs& t, int mode, int lvl, cudaStream_t stream);

}  // namespace pm
