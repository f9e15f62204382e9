// internal.h - pieces of the C ABI implementation shared between its translation units.
#pragma once

#include <cuda_runtime.h>

#include "kernels.h"
#include "planner.h"

namespace emoe {

// Runs one phase plan once on the current device: builds and uploads its descriptor
// tables, launches the copy kernels on `st`, synchronises `st`, frees the tables.
// Returns EMOE_ERR_DEVICE_TIMEOUT if a bounded device wait expired.
emoe_status_t run_phase_once(const PhasePlan &pp, const RankPtrs &ptrs, cudaStream_t st);

}  // namespace emoe
