// Launch wrappers implemented in the .cu files (kept free of kernel code so that host-only
// translation units can include it).
#pragma once
#include <cuda_runtime.h>

#include "pl_internal.h"

namespace pl {

// register (ld/st) executor
cudaError_t launch_exec(int dtype, const ExecParams& P, int grid, int threads, cudaStream_t stream);
int exec_max_ctas_per_sm(int dtype, int threads);
int exec_max_threads();

// TMA (bulk-copy, shared-memory ring) executor
cudaError_t launch_exec_tma(int dtype, const ExecParams& P, int grid, cudaStream_t stream);
int exec_tma_max_ctas_per_sm(int dtype, int stages, uint32_t stage_bytes);
// threads per CTA of the two variants: general (16 consumer warps) and pipelined reduce (12)
int exec_tma_threads(bool pipelined);
size_t exec_tma_smem_bytes(int stages, uint32_t stage_bytes);

// packet executor (latency path): rank = cluster of ctas_per_rank CTAs
cudaError_t launch_exec_packet(int dtype, const PacketParams& P, int threads, bool overlap, cudaStream_t stream);
int exec_packet_max_groups(int dtype, int ctas_per_rank, int threads);
int exec_packet_max_units_per_thread();
int exec_packet_max_threads();

}  // namespace pl
