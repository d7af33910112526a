// Internal: what multi.cu needs of a plan (defined in api.cu) without seeing its layout.
#pragma once
#include "schedule.h"

struct sparbit_plan_s;

namespace spb {
const Schedule* plan_schedule(const sparbit_plan_s* p);
bool plan_is_variable(const sparbit_plan_s* p);
// Stores "<what>: <cudaGetErrorString>" for sparbit_last_cuda_error(); returns SPARBIT_ERR_CUDA.
int record_cuda_error(int cuda_error, const char* what);
}  // namespace spb
