// Tensor-core (tcgen05 / TMEM / TMA) grouped GEMMs of the step -- placeholder plan while the SIMT path is brought up.
#pragma once
#include <vector>
#include "../../include/ngalore.h"
#include "common.cuh"
namespace ngalore {
struct TcPlan { size_t device_bytes = 0; };
inline ngalore_status tc_plan_create(TcPlan&, const std::vector<MatDesc>&, const MatDesc*, int, int) { return NGALORE_OK; }
inline void tc_plan_destroy(TcPlan&) {}
inline ngalore_status tc_project(TcPlan&, const MatDesc*, Ctrl*, const uint16_t* const*, bool, cudaStream_t, int64_t*) { return NGALORE_ERR_INVALID_ARG; }
inline ngalore_status tc_backproject(TcPlan&, const MatDesc*, Ctrl*, const Hyper*, float* const*, bool, cudaStream_t, int64_t*) { return NGALORE_ERR_INVALID_ARG; }
}  // namespace ngalore
