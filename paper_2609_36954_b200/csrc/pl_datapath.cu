// Datapath: one persistent kernel; CTA q interprets op queue q.
//
// Per op: wait (acquire) on the op's flags -> body (copy / reduce / copy-reduce with 128-bit
// accesses, fp32 accumulation in ascending source order, Sec. 3.3 Eq. "rank-order") ->
// signal (release).  Flags are 64-bit counters that only grow: execute number e expects
// e * need signals, so nothing is reset between executes and the epoch lives on the device
// (Sec. 4.2 keeps a persistent epoch for the same reason).  Every wait is bounded by a
// globaltimer limit; on expiry the CTA records a status, raises the abort word that every
// waiter also polls, and the kernel returns normally.
#include <cuda_bf16.h>
#include <cuda_runtime.h>

#include <algorithm>

#include "pl_device.cuh"
#include "pl_internal.h"
#include "pl_kernels.h"

namespace pl {
namespace {

using namespace dev;

constexpr int kMaxThreads = 512;

// ---- op bodies (register path: unrolled 128-bit loads, then stores) -----------------------
__device__ __forceinline__ void body_copy(char* dst, const char* src, uint64_t bytes, int tid, int nthr) {
  const uint64_t n = bytes >> 4;
  constexpr int U = 8;
  uint64_t i = tid;
  for (; i + (uint64_t)(U - 1) * nthr < n; i += (uint64_t)U * nthr) {
    uint4 v[U];
#pragma unroll
    for (int u = 0; u < U; ++u) v[u] = ld16(src + ((i + (uint64_t)u * nthr) << 4));
#pragma unroll
    for (int u = 0; u < U; ++u) st16(dst + ((i + (uint64_t)u * nthr) << 4), v[u]);
  }
  for (; i < n; i += nthr) st16(dst + (i << 4), ld16(src + (i << 4)));
}

// The same bytes to the same offset of every rank's output (a pushed all-gather contribution).
__device__ __forceinline__ void body_copy_bcast(const ExecParams& P, uint64_t dst_off, const char* src, uint64_t bytes,
                                                int tid, int nthr) {
  const uint64_t n = bytes >> 4;
  constexpr int U = 4;
  for (uint64_t i = tid; i < n; i += (uint64_t)U * nthr) {
    uint4 v[U];
#pragma unroll
    for (int u = 0; u < U; ++u)
      if (i + (uint64_t)u * nthr < n) v[u] = ld16(src + ((i + (uint64_t)u * nthr) << 4));
    for (int k = 0; k < P.n_ranks; ++k) {
      char* d = static_cast<char*>(P.base[kSlotOut + k]) + dst_off;
#pragma unroll
      for (int u = 0; u < U; ++u)
        if (i + (uint64_t)u * nthr < n) st16(d + ((i + (uint64_t)u * nthr) << 4), v[u]);
    }
  }
}

// Add NB same-typed sources (ascending) for U units at once: all loads first, then the adds.
template <int DT, int NB, int U>
__device__ __forceinline__ void accumulate_batch(Acc<DT> (&acc)[U], const char* const* src, const uint64_t (&off)[U]) {
  uint4 q[U][NB];
#pragma unroll
  for (int u = 0; u < U; ++u)
#pragma unroll
    for (int s = 0; s < NB; ++s) q[u][s] = ld16(src[s] + off[u]);
#pragma unroll
  for (int u = 0; u < U; ++u)
#pragma unroll
    for (int s = 0; s < NB; ++s) {
      if constexpr (DT == PL_BF16) acc[u].add_bf16(q[u][s]);
      else acc[u].add(q[u][s]);
    }
}

// Reduce U units (unit index first + u*stride) from ns sources and store the result.
template <int DT, int U, bool HOOK>
__device__ __forceinline__ void reduce_units(const ExecParams& P, const char* const* s_src, int ns, char* dst,
                                             uint64_t dst_off, bool bcast, uint64_t first, uint64_t stride,
                                             uint64_t dst_slot, bool final_op) {
  Acc<DT> acc[U];
  uint64_t off[U];
#pragma unroll
  for (int u = 0; u < U; ++u) {
    acc[u].zero();
    off[u] = (first + (uint64_t)u * stride) << 4;
  }
  int s = 0;
#pragma unroll 1
  for (; s + 4 <= ns; s += 4) accumulate_batch<DT, 4, U>(acc, s_src + s, off);
  if (s + 2 <= ns) { accumulate_batch<DT, 2, U>(acc, s_src + s, off); s += 2; }
  if (s < ns) accumulate_batch<DT, 1, U>(acc, s_src + s, off);
  if constexpr (HOOK) {
    if (final_op) {  // the processing phase: scale, second operand, output type
#pragma unroll
      for (int u = 0; u < U; ++u) store_final_unit<DT>(P, acc[u], dst_slot, dst_off, bcast, first + (uint64_t)u * stride);
      return;
    }
  }
#pragma unroll
  for (int u = 0; u < U; ++u) {
    uint4 r;
    if constexpr (DT == PL_BF16) r = acc[u].to_bf16(P.out_scale);
    else r = acc[u].result(P.out_scale);
    if (!bcast) {
      st16(dst + off[u], r);
    } else {
      for (int k = 0; k < P.n_ranks; ++k) st16(static_cast<char*>(P.base[kSlotOut + k]) + dst_off + off[u], r);
    }
  }
}

// REDUCE with n same-typed sources -> element-typed destination (optionally replicated to
// every rank's output).  s_src holds the resolved source pointers in shared memory.
template <int DT, bool HOOK>
__device__ __forceinline__ void body_reduce(const ExecParams& P, const DevOp& op, const char* const* s_src, char* dst, int tid,
                                            int nthr) {
  constexpr int U = 2;
  const uint64_t dst_slot = op.dst >> 48;
  const bool final_op = op.flags & kFinal;
  const uint64_t n_units = op.count / Acc<DT>::kElems;  // 16 bytes of every operand each
  const bool bcast = op.flags & kDstBcast;
  const uint64_t dst_off = op.dst & 0xFFFFFFFFFFFFull;
  const int ns = op.n_src;
  uint64_t base = tid;
  for (; base + (uint64_t)(U - 1) * nthr < n_units; base += (uint64_t)U * nthr)
    reduce_units<DT, U, HOOK>(P, s_src, ns, dst, dst_off, bcast, base, nthr, dst_slot, final_op);
  for (; base < n_units; base += nthr) reduce_units<DT, 1, HOOK>(P, s_src, ns, dst, dst_off, bcast, base, nthr, dst_slot, final_op);
}

// COPY_REDUCE: dst = a + b where a and/or b may hold fp32 partials of a bf16 reduction and
// dst may be a partial too.  For fp32 / int32 data every operand has the element type.
// Final hop of a travelling sum in a hooked schedule: dst = process(a + b).
template <int DT>
__device__ __forceinline__ void body_copy_reduce_final(const ExecParams& P, const DevOp& op, const char* const* s_src,
                                                       int tid, int nthr) {
  if constexpr (DT == PL_BF16 || DT == PL_F32) {
    const uint64_t n_units = op.count / Acc<DT>::kElems;
    const char* a = s_src[0];
    const char* b = s_src[1];
    const bool ap = op.src_f32_mask & 1u, bp = op.src_f32_mask & 2u;
    const uint64_t dst_slot = op.dst >> 48, dst_off = op.dst & 0xFFFFFFFFFFFFull;
    for (uint64_t i = tid; i < n_units; i += nthr) {
      Acc<DT> acc;
      acc.zero();
      if constexpr (DT == PL_BF16) {
        if (ap) acc.add_f32(ld16(a + (i << 5)), ld16(a + (i << 5) + 16)); else acc.add_bf16(ld16(a + (i << 4)));
        if (bp) acc.add_f32(ld16(b + (i << 5)), ld16(b + (i << 5) + 16)); else acc.add_bf16(ld16(b + (i << 4)));
      } else {
        if (ap) acc.add_pair(ld16(a + (i << 5)), ld16(a + (i << 5) + 16)); else acc.add(ld16(a + (i << 4)));
        if (bp) acc.add_pair(ld16(b + (i << 5)), ld16(b + (i << 5) + 16)); else acc.add(ld16(b + (i << 4)));
      }
      store_final_unit<DT>(P, acc, dst_slot, dst_off, false, i);
    }
  }
}

template <int DT>
__device__ __forceinline__ void body_copy_reduce(const ExecParams& P, const DevOp& op, const char* const* s_src, char* dst,
                                                 int tid, int nthr) {
  const uint64_t n_units = op.count / Acc<DT>::kElems;
  const char* a = s_src[0];
  const char* b = s_src[1];
  if constexpr (DT == PL_I32) {
    constexpr int U = 4;
    for (uint64_t base = tid; base < n_units; base += (uint64_t)U * nthr) {
      uint4 qa[U], qb[U];
#pragma unroll
      for (int u = 0; u < U; ++u) {
        const uint64_t i = base + (uint64_t)u * nthr;
        if (i < n_units) { qa[u] = ld16(a + (i << 4)); qb[u] = ld16(b + (i << 4)); }
      }
#pragma unroll
      for (int u = 0; u < U; ++u) {
        const uint64_t i = base + (uint64_t)u * nthr;
        if (i < n_units) {
          Acc<DT> acc;
          acc.zero();
          acc.add(qa[u]);
          acc.add(qb[u]);
          st16(dst + (i << 4), acc.result(P.out_scale));
        }
      }
    }
  } else if constexpr (DT == PL_F32) {
    // operands are fp32 vectors (16 B per unit) or (sum, correction) pairs (32 B per unit)
    const bool ap = op.src_f32_mask & 1u, bp = op.src_f32_mask & 2u, dp = op.flags & kDstF32;
    constexpr int U = 2;
    for (uint64_t base = tid; base < n_units; base += (uint64_t)U * nthr) {
      uint4 qa[U][2], qb[U][2];
#pragma unroll
      for (int u = 0; u < U; ++u) {
        const uint64_t i = base + (uint64_t)u * nthr;
        if (i < n_units) {
          if (ap) { qa[u][0] = ld16(a + (i << 5)); qa[u][1] = ld16(a + (i << 5) + 16); }
          else qa[u][0] = ld16(a + (i << 4));
          if (bp) { qb[u][0] = ld16(b + (i << 5)); qb[u][1] = ld16(b + (i << 5) + 16); }
          else qb[u][0] = ld16(b + (i << 4));
        }
      }
#pragma unroll
      for (int u = 0; u < U; ++u) {
        const uint64_t i = base + (uint64_t)u * nthr;
        if (i < n_units) {
          Acc<PL_F32> acc;
          acc.zero();
          if (ap) acc.add_pair(qa[u][0], qa[u][1]); else acc.add(qa[u][0]);
          if (bp) acc.add_pair(qb[u][0], qb[u][1]); else acc.add(qb[u][0]);
          if (dp) {
            st16(dst + (i << 5), acc.sums());
            st16(dst + (i << 5) + 16, acc.corrections());
          } else {
            st16(dst + (i << 4), acc.result(P.out_scale));
          }
        }
      }
    }
  } else {
    const bool a32 = op.src_f32_mask & 1u, b32 = op.src_f32_mask & 2u, d32 = op.flags & kDstF32;
    constexpr int U = 2;
    for (uint64_t base = tid; base < n_units; base += (uint64_t)U * nthr) {
      uint4 qa[U][2], qb[U][2];
#pragma unroll
      for (int u = 0; u < U; ++u) {
        const uint64_t i = base + (uint64_t)u * nthr;
        if (i < n_units) {
          if (a32) { qa[u][0] = ld16(a + (i << 5)); qa[u][1] = ld16(a + (i << 5) + 16); }
          else qa[u][0] = ld16(a + (i << 4));
          if (b32) { qb[u][0] = ld16(b + (i << 5)); qb[u][1] = ld16(b + (i << 5) + 16); }
          else qb[u][0] = ld16(b + (i << 4));
        }
      }
#pragma unroll
      for (int u = 0; u < U; ++u) {
        const uint64_t i = base + (uint64_t)u * nthr;
        if (i < n_units) {
          Acc<PL_BF16> acc;
          acc.zero();
          if (a32) acc.add_f32(qa[u][0], qa[u][1]); else acc.add_bf16(qa[u][0]);
          if (b32) acc.add_f32(qb[u][0], qb[u][1]); else acc.add_bf16(qb[u][0]);
          if (d32) {
            uint4 lo = make_uint4(__float_as_uint(acc.v[0]), __float_as_uint(acc.v[1]), __float_as_uint(acc.v[2]), __float_as_uint(acc.v[3]));
            uint4 hi = make_uint4(__float_as_uint(acc.v[4]), __float_as_uint(acc.v[5]), __float_as_uint(acc.v[6]), __float_as_uint(acc.v[7]));
            st16(dst + (i << 5), lo);
            st16(dst + (i << 5) + 16, hi);
          } else {
            st16(dst + (i << 4), acc.to_bf16(P.out_scale));
          }
        }
      }
    }
  }
}

// ---- the executor -------------------------------------------------------------------------
struct OpSlot {
  DevOp op;
  const char* src[PL_MAX_SRC];
  DevWait wait[PL_MAX_WAITS];
};

// BC: the variant that also runs broadcast copies (pushed all-gather, broadcast).  It is a
// kernel of its own because the mere presence of that body in the function changed the code
// generated for the reduce loops (one-shot all-reduce of 8 MiB per rank: 71 -> 88 us);
// schedules with broadcast copies hold no reduce ops, schedules with reduce ops run BC = false.
// HOOK: the variant for schedules with a processing phase beyond the scale (PL_HOOK_*): its
// final reduce ops add the second operand and / or keep fp32.  A kernel of its own for the
// same reason as BC: the plain variants keep the code they have.
// DBUF: the variant for staged schedules with two staging buffers (PL_OPT_STAGE_AHEAD): flag set
// and staging buffer follow the parity of a launch counter taken at entry, and the leading
// stage ops of a queue run before the kernel waits for the launch in front of it.
template <int DT, bool BC, bool HOOK = false, bool DBUF = false>
__global__ void __launch_bounds__(kMaxThreads) pl_exec_kernel(const __grid_constant__ ExecParams P) {
  __shared__ OpSlot s_slot[2];
  __shared__ int s_abort[2];  // indexed by iteration parity: written during wait i, read after barrier i
  __shared__ unsigned long long s_launch;
  const int tid = threadIdx.x, nthr = blockDim.x, q = blockIdx.x;
  const uint32_t nq = P.n_queues;
  // every CTA reads the epoch before it reports completion, and the epoch word is only
  // advanced after all CTAs reported, so all of them see the same value; a schedule without
  // flags needs no epoch at all
  const bool has_flags = P.flags != nullptr;
  if constexpr (!DBUF) pdl_launch_dependents();
  if (tid == 0) s_abort[0] = s_abort[1] = 0;
  bool aborted = false;
  unsigned long long scratch_shift = 0ull;       // DBUF: distance to this launch's staging buffer
  const unsigned long long* flag_base = P.flags;  // DBUF: this launch's flag set

  // descriptor fetch by warp 0: lanes 0-3 carry the op, lane k source k and wait entry k
  auto fetch = [&](uint32_t i, uint4& r_op, uint64_t& r_src, DevWait& r_wait) {
    const uint64_t at = (uint64_t)i * nq + q;  // op i of this queue
    if (tid < 4) r_op = reinterpret_cast<const uint4*>(P.ops + at)[tid];
    if (tid < (int)P.src_stride) r_src = P.srcs[at * P.src_stride + tid];
    if (tid < (int)P.wait_stride) r_wait = P.waits[at * P.wait_stride + tid];
  };
  auto stash = [&](int slot, const uint4& r_op, uint64_t r_src, const DevWait& r_wait) {
    if (tid < 4) reinterpret_cast<uint4*>(&s_slot[slot].op)[tid] = r_op;
    if (tid < (int)P.src_stride) s_slot[slot].src[tid] = DBUF ? resolve(P, r_src, scratch_shift) : resolve(P, r_src);
    if (tid < (int)P.wait_stride) s_slot[slot].wait[tid] = r_wait;
  };

  uint4 r_op = make_uint4(0, 0, 0, 0);
  uint64_t r_src = 0;
  DevWait r_wait = {0, 0};
  if (tid < 32) fetch(0, r_op, r_src, r_wait);  // descriptors are immutable: fetched before the wait below
  unsigned long long epoch;
  bool waited = !DBUF;  // DBUF: griddepcontrol.wait is still to come (before the first op that is not an early stage op)
  if constexpr (DBUF) {
    // Launch number: every CTA of launch i takes its ticket before it lets launch i+1 start, so
    // ticket / grid is i for all of them (also under graph replay).  Parity picks the flag set
    // and the staging buffer; a set is used by every second launch, hence its own epoch i / 2.
    if (tid == 0) s_launch = atomicAdd(P.epoch + 2, 1ull) / gridDim.x;
    __syncthreads();
    const unsigned long long launch = s_launch;
    epoch = (launch >> 1) + 1ull;
    if (launch & 1ull) {
      scratch_shift = P.scratch_half;
      flag_base = P.flags + P.n_flags;
    }
  } else {
    pdl_wait();
    epoch = has_flags ? *reinterpret_cast<volatile unsigned long long*>(P.epoch) + 1ull : 0ull;
  }
  if (tid < 32) stash(0, r_op, r_src, r_wait);
  __syncthreads();
  // the first descriptor tells how many ops the queue holds (a placeholder marks an empty one)
  const uint32_t n_ops = s_slot[0].op.kind == kNopKind ? 0u : s_slot[0].op.remaining + 1u;

  for (uint32_t i = 0; i < n_ops; ++i) {
    const int slot = i & 1;
    OpSlot& S = s_slot[slot];
    if constexpr (DBUF) {
      // everything but the leading early-stage ops runs after the launch in front has completed;
      // only then may the launch behind this one start (it shares this launch's other buffer)
      if (!waited && !(S.op.flags & kStageAhead)) {
        pdl_wait();
        pdl_launch_dependents();
        waited = true;
      }
    }
    if (tid < 32) {
      // ---- wait: lane k polls wait entry k (acquire), bounded by the time limit
      const uint32_t nw = S.op.n_wait;
      if (tid < (int)nw) {
        const DevWait w = S.wait[tid];
        const unsigned long long need = epoch * (unsigned long long)w.need;
        const unsigned long long* fp = flag_base + w.flag;
        unsigned long long seen = ld_acquire_u64(fp);
        if (seen < need) {
          const unsigned long long t0 = globaltimer_ns();
          uint32_t spins = 0;
          while ((seen = ld_acquire_u64(fp)) < need) {
            if ((++spins & 63u) == 0) {
              if (ld_volatile_s32(P.status + 8)) { s_abort[slot] = 1; break; }
              if (globaltimer_ns() - t0 > P.timeout_ns) {
                record_timeout(P, q, S.op.topo, w.flag, need, seen);
                s_abort[slot] = 1;
                break;
              }
            }
          }
        }
      }
      __syncwarp();
    }
    __syncthreads();  // descriptor + satisfied waits visible to the CTA; previous body finished
    if (s_abort[slot]) { aborted = true; break; }
    const bool has_next = i + 1 < n_ops;
    if (tid < 32 && has_next) fetch(i + 1, r_op, r_src, r_wait);

    const DevOp& op = S.op;
    if (P.trace && tid == 0) P.trace[2ull * op.topo] = globaltimer_ns();  // waits satisfied
    char* const op_dst = DBUF ? resolve(P, op.dst, scratch_shift) : resolve(P, op.dst);
    if (op.kind == PL_OP_COPY) {
      if constexpr (BC) {
        if (op.flags & kDstBcast) body_copy_bcast(P, op.dst & 0xFFFFFFFFFFFFull, S.src[0], op.count, tid, nthr);
        else body_copy(op_dst, S.src[0], op.count, tid, nthr);
      } else {
        body_copy(op_dst, S.src[0], op.count, tid, nthr);
      }
    } else if (op.kind == PL_OP_REDUCE) {
      if constexpr (DT != PL_U8) body_reduce<DT, HOOK>(P, op, S.src, op_dst, tid, nthr);
    } else {
      if constexpr (DT != PL_U8) {
        if (HOOK && (op.flags & kFinal)) body_copy_reduce_final<DT>(P, op, S.src, tid, nthr);
        else body_copy_reduce<DT>(P, op, S.src, op_dst, tid, nthr);
      }
    }

    if (op.signal != kNoFlag || P.trace) {
      __syncthreads();  // every thread's writes are done
      if (tid == 0 && P.trace) P.trace[2ull * op.topo + 1] = globaltimer_ns();
      if (tid == 0 && op.signal != kNoFlag) {
        // the release is cumulative: it covers the other threads' stores, which this thread
        // observed through the barrier above
        red_release_add_u64(const_cast<unsigned long long*>(flag_base) + op.signal, 1ull);
        if (op.signal2 != kNoFlag) red_release_add_u64(const_cast<unsigned long long*>(flag_base) + op.signal2, 1ull);
      }
    }
    if (tid < 32 && has_next) {
      stash(slot ^ 1, r_op, r_src, r_wait);
      __syncwarp();
    }
  }

  if constexpr (DBUF) {
    if (!waited) {  // a queue of early stage ops only (or an empty one): still ordered behind the launch in front
      pdl_wait();
      pdl_launch_dependents();
    }
  }
  __syncthreads();
  if (tid == 0 && !aborted && has_flags && !DBUF) {
    // last CTA to finish advances the epoch for the next execute
    const unsigned long long prev = atomicAdd(P.epoch + 1, 1ull);
    if (prev == (unsigned long long)gridDim.x - 1ull) {
      P.epoch[1] = 0ull;
      __threadfence();
      *reinterpret_cast<volatile unsigned long long*>(P.epoch) = epoch;
    }
  }
}

template <int DT, bool BC, bool HOOK = false, bool DBUF = false>
cudaError_t launch_t(const ExecParams& P, int grid, int threads, cudaStream_t stream) {
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = dim3((unsigned)grid);
  cfg.blockDim = dim3((unsigned)threads);
  cfg.stream = stream;
  cudaLaunchAttribute attr[1];
  attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  attr[0].val.programmaticStreamSerializationAllowed = 1;
  cfg.attrs = attr;
  cfg.numAttrs = P.overlap_launch ? 1 : 0;
  return cudaLaunchKernelEx(&cfg, pl_exec_kernel<DT, BC, HOOK, DBUF>, P);
}

}  // namespace

cudaError_t launch_exec(int dtype, const ExecParams& P, int grid, int threads, cudaStream_t stream) {
  if (P.hook) {  // float schedules with reduce ops only (checked at build)
    switch (dtype) {
      case PL_BF16: return launch_t<PL_BF16, false, true>(P, grid, threads, stream);
      case PL_F32: return launch_t<PL_F32, false, true>(P, grid, threads, stream);
      default: return cudaErrorInvalidValue;
    }
  }
  if (P.stage_ahead) {  // staged schedules: copies and plain reduces, no broadcast copies, no hooks (checked at build)
    switch (dtype) {
      case PL_BF16: return launch_t<PL_BF16, false, false, true>(P, grid, threads, stream);
      case PL_F32: return launch_t<PL_F32, false, false, true>(P, grid, threads, stream);
      case PL_I32: return launch_t<PL_I32, false, false, true>(P, grid, threads, stream);
      default: return launch_t<PL_U8, false, false, true>(P, grid, threads, stream);
    }
  }
  if (P.bcast_copies) {
    switch (dtype) {
      case PL_BF16: return launch_t<PL_BF16, true>(P, grid, threads, stream);
      case PL_F32: return launch_t<PL_F32, true>(P, grid, threads, stream);
      case PL_I32: return launch_t<PL_I32, true>(P, grid, threads, stream);
      default: return launch_t<PL_U8, true>(P, grid, threads, stream);
    }
  }
  switch (dtype) {
    case PL_BF16: return launch_t<PL_BF16, false>(P, grid, threads, stream);
    case PL_F32: return launch_t<PL_F32, false>(P, grid, threads, stream);
    case PL_I32: return launch_t<PL_I32, false>(P, grid, threads, stream);
    default: return launch_t<PL_U8, false>(P, grid, threads, stream);
  }
}

namespace {
template <int DT>
int occupancy_both(int threads) {
  // capacity that holds for whichever variant a schedule launches
  int a = 0, b = 0, c = 1 << 30;
  if (cudaOccupancyMaxActiveBlocksPerMultiprocessor(&a, pl_exec_kernel<DT, true>, threads, 0) != cudaSuccess ||
      cudaOccupancyMaxActiveBlocksPerMultiprocessor(&b, pl_exec_kernel<DT, false>, threads, 0) != cudaSuccess) {
    cudaGetLastError();
    return 0;
  }
  if constexpr (DT == PL_BF16 || DT == PL_F32) {
    if (cudaOccupancyMaxActiveBlocksPerMultiprocessor(&c, pl_exec_kernel<DT, false, true>, threads, 0) != cudaSuccess) {
      cudaGetLastError();
      return 0;
    }
  }
  int d = 0;
  if (cudaOccupancyMaxActiveBlocksPerMultiprocessor(&d, pl_exec_kernel<DT, false, false, true>, threads, 0) != cudaSuccess) {
    cudaGetLastError();
    return 0;
  }
  return std::min(std::min(a, b), std::min(c, d));
}
}  // namespace

int exec_max_ctas_per_sm(int dtype, int threads) {
  switch (dtype) {
    case PL_BF16: return occupancy_both<PL_BF16>(threads);
    case PL_F32: return occupancy_both<PL_F32>(threads);
    case PL_I32: return occupancy_both<PL_I32>(threads);
    default: return occupancy_both<PL_U8>(threads);
  }
}

int exec_max_threads() { return kMaxThreads; }

}  // namespace pl
