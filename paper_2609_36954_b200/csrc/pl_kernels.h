// Launch wrappers implemented in the .cu files (kept free of kernel code so that host-only
// translation units can include it).
#pragma once
#include <cuda_runtime.h>

#include "pl_internal.h"

namespace pl {

cudaError_t launch_exec(int dtype, const ExecParams& P, int grid, int threads, cudaStream_t stream);
int exec_max_ctas_per_sm(int dtype, int threads);
int exec_max_threads();

}  // namespace pl
