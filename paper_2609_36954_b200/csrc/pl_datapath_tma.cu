// Throughput datapath: the op-queue executor built around bulk asynchronous copies (TMA).
//
// One CTA per op queue, warp specialised:
//   warps 0, 1  producers  both walk the queue, wait on every op's flags (acquire, bounded) and
//                     cut the op into stages; producer p fills the ring slots of the stages
//                     with number n = p (mod 2) with cp.async.bulk loads (one per source),
//                     running ahead of the consumers across op boundaries (Algorithm 2 of the
//                     paper: prime / steady / drain, here as a free-running ring with full /
//                     empty mbarriers).  Two of them because issuing is what a producer spends
//                     its time on: the bulk loads of one warp are accepted one at a time,
//                     60-70 ns each, so the 8 loads of an 8-source stage plus the stage's
//                     bookkeeping (about 1 us) took as long as HBM needs to deliver its 48 KiB;
//   warp 2  copier    for COPY stages: one bulk store shared -> global per stage (R stores
//                     for a broadcast copy), no registers touched by the payload;
//   warps 3..  consumers (16, or 12 in the variant for plain reduce schedules)  for REDUCE /
//                     COPY_REDUCE stages: read the source tiles from shared memory 16 bytes
//                     at a time, accumulate in fp32 in ascending source order, store the
//                     result with 128-bit global stores.
// A stage descriptor travels with every slot.  The last stage of an op carries its signal:
// the warps that wrote report on an mbarrier, then one thread fences and does the release
// increment.  Every wait (flag, full, empty, done) is bounded; on expiry the CTA records a
// status, raises the abort word and leaves after draining its own copies.
#include <cuda_bf16.h>
#include <cuda_runtime.h>

#include <algorithm>
#include <atomic>

#include "pl_device.cuh"
#include "pl_internal.h"
#include "pl_kernels.h"
#include "pl_ptx.cuh"

namespace pl {
namespace {

using namespace dev;

// Consumer warps per CTA (template parameter CW of the kernel): 16 in general; 12 for
// schedules made of plain reduce stages only, where the software-pipelined path below keeps two
// stages of operands in registers (128 registers per thread need the smaller CTA).
constexpr int kWarpsGeneral = 16;
constexpr int kWarpsPipelined = 12;
constexpr int kProducers = 2;  // producer warps; the copier is warp kProducers, consumers follow
constexpr int kMaxStages = 8;
constexpr uint32_t kEnd = 0xFFFFFFFFu;
constexpr uint32_t kLastOfOp = 0x100u;  // stage flag (above the DevOp flag bits)
constexpr uint32_t kAuxInSlot = 0x200u;  // stage flag: the second operand's tile sits in the slot behind the sources
// Stage flag of a final op with R destinations (fused all-reduce with a processing phase): the
// consumers leave the results in the slot at res_off (+ k * res_stride for rank k when the
// results differ per rank) and the copier ships them with bulk stores.
constexpr uint32_t kResInSlot = 0x400u;
constexpr int kCtrlBytes = 1024;        // barriers + stage descriptors ahead of the slots

struct StageDesc {
  uint32_t kind;   // pl_op_kind_t or kEnd
  uint32_t n_src;
  uint32_t units;  // 16-byte units of the element type in this stage (COPY: bytes / 16)
  uint32_t ucap;   // unit capacity of a slot for this op (tile k starts at a multiple of it)
  uint32_t pmask;  // sources that hold partials (twice as wide)
  uint32_t flags;  // kDstF32 | kDstBcast | kLastOfOp
  uint32_t signal, signal2;
  char* dst;       // destination of this stage
  uint64_t dst_off;  // byte offset inside every rank's output (broadcast destinations)
  uint32_t topo;   // the op's topological index (trace)
  uint32_t dst_slot;  // pointer-table slot of the destination (hooked schedules: finds the second operand)
};
static_assert(sizeof(StageDesc) == 56, "StageDesc layout");
// kResInSlot stages: the result region starts right behind the n_src source tiles; with a second
// operand (PL_HOOK_RESIDUAL) it is one tile per rank (rank k's result over rank k's operand
// tile), otherwise one region of 32 bytes per unit.
__device__ __forceinline__ uint32_t res_off(const StageDesc& d) { return d.ucap * 16u * d.n_src; }
__device__ __forceinline__ uint32_t res_stride(const ExecParams& P, const StageDesc& d) {
  return (P.hook & PL_HOOK_RESIDUAL) ? d.ucap * 16u : 0u;
}

struct Ctrl {
  uint64_t full[kMaxStages];
  uint64_t empty[kMaxStages];
  // consumer warps that finished writing the last stage of an op.  One barrier per slot: a
  // fast warp can be a whole stage ahead of a slow one, and arrivals for two different
  // stages must never meet on one barrier.
  uint64_t done[kMaxStages];
  int abort;
  int pad;
  unsigned long long launch;  // double-buffered staging: number of this launch (taken at entry by thread 0)
  int q;                      // SM-window launches: the queue this CTA claimed (-1: its SM sits out)
  StageDesc desc[kMaxStages];
};
static_assert(sizeof(Ctrl) <= kCtrlBytes, "control block too large");

// Bounded mbarrier wait.  Returns false when the CTA is aborting or the time limit passed.
// Waits inside a CTA get twice the limit of a flag wait: when a dependency never arrives, the
// warps starved behind the producer started waiting earlier than the producer itself, and the
// record should name the flag (the cause), not a starved barrier.
__device__ __forceinline__ bool wait_bar(const ExecParams& P, Ctrl* c, uint64_t* bar, uint32_t parity) {
  if (ptx::mbar_try_wait(bar, parity)) return true;
  const unsigned long long t0 = globaltimer_ns();
  for (uint32_t spins = 1;; ++spins) {
    if (ptx::mbar_try_wait(bar, parity)) return true;
    if ((spins & 255u) == 0) {
      if (*reinterpret_cast<volatile int*>(&c->abort)) return false;
      if (globaltimer_ns() - t0 > 2ull * P.timeout_ns + 1000000ull) {
        record_timeout(P, c->q, 0xFFFFFFFFu, 0xFFFFFFFFu, parity, 0);
        *reinterpret_cast<volatile int*>(&c->abort) = 1;
        return false;
      }
    }
  }
}

__device__ __forceinline__ uint4 lds16(const unsigned char* p) {
  uint4 v;
  asm volatile("ld.shared.v4.u32 {%0,%1,%2,%3}, [%4];" : "=r"(v.x), "=r"(v.y), "=r"(v.z), "=r"(v.w) : "r"(ptx::smem_u32(p)));
  return v;
}

// Consumer work for one stage of a REDUCE / COPY_REDUCE op.
template <int DT, int CW, bool HOOK>
__device__ __forceinline__ void consume_stage(const ExecParams& P, const StageDesc& d, const unsigned char* slot, int ctid) {
  const uint32_t units = d.units, ns = d.n_src, pmask = d.pmask;
  const uint32_t tile = d.ucap * 16u;  // bytes of an element-typed tile; partial tiles are twice that
  const bool dpart = d.flags & kDstF32, bcast = d.flags & kDstBcast;
  const bool final_op = HOOK && (d.flags & kFinal);
  for (uint32_t u = ctid; u < units; u += 32 * CW) {
    Acc<DT> acc;
    acc.zero();
    if (pmask == 0) {
      // all sources element-typed: loads of four sources at a time, then the adds (ascending)
      const unsigned char* p = slot + (size_t)u * 16u;
      uint32_t s = 0;
      for (; s + 4 <= ns; s += 4) {
        uint4 q0 = lds16(p), q1 = lds16(p + tile), q2 = lds16(p + 2 * tile), q3 = lds16(p + 3 * tile);
        p += 4 * (size_t)tile;
        if constexpr (DT == PL_BF16) { acc.add_bf16(q0); acc.add_bf16(q1); acc.add_bf16(q2); acc.add_bf16(q3); }
        else { acc.add(q0); acc.add(q1); acc.add(q2); acc.add(q3); }
      }
      for (; s < ns; ++s) {
        uint4 q = lds16(p);
        p += tile;
        if constexpr (DT == PL_BF16) acc.add_bf16(q);
        else acc.add(q);
      }
    } else {
      const unsigned char* base = slot;
      for (uint32_t s = 0; s < ns; ++s) {
        const bool part = (pmask >> s) & 1u;
        if constexpr (DT == PL_I32) {
          acc.add(lds16(base + (size_t)u * 16u));
          base += tile;
        } else if (part) {
          const uint4 lo = lds16(base + (size_t)u * 32u), hi = lds16(base + (size_t)u * 32u + 16u);
          if constexpr (DT == PL_BF16) acc.add_f32(lo, hi);
          else acc.add_pair(lo, hi);
          base += 2 * (size_t)tile;
        } else {
          const uint4 q = lds16(base + (size_t)u * 16u);
          if constexpr (DT == PL_BF16) acc.add_bf16(q);
          else acc.add(q);
          base += tile;
        }
      }
    }
    if (final_op) {
      // processing phase of a hooked schedule: scale, second operand, output type; one store
      // per destination (the results may differ per rank, so nothing leaves through the slot)
      if constexpr (HOOK && (DT == PL_BF16 || DT == PL_F32)) {
        if (d.flags & kResInSlot) {
          // R destinations: results go into the slot, the copier stores them.  With a second
          // operand (one tile per rank, brought by the producer) rank k's result replaces unit u
          // of rank k's operand tile, which only this thread reads; otherwise one result of 32
          // bytes per unit (fp32 output) goes to a region of its own behind the sources.
          unsigned char* res = const_cast<unsigned char*>(slot) + res_off(d);
          const uint32_t stride = res_stride(P, d);
          if (stride) {
            for (int k = 0; k < P.n_ranks; ++k) {
              unsigned char* at = res + (size_t)k * stride + (size_t)u * 16u;
              uint4 lo, hi;
              final_value<DT>(acc, P.out_scale, P.hook, lds16(at), lo, hi);
              asm volatile("st.shared.v4.u32 [%0], {%1,%2,%3,%4};" ::"r"(ptx::smem_u32(at)), "r"(lo.x), "r"(lo.y), "r"(lo.z), "r"(lo.w) : "memory");
            }
          } else {
            uint4 lo, hi = make_uint4(0, 0, 0, 0);
            final_value<DT>(acc, P.out_scale, P.hook, make_uint4(0, 0, 0, 0), lo, hi);
            unsigned char* at = res + (size_t)u * 32u;
            asm volatile("st.shared.v4.u32 [%0], {%1,%2,%3,%4};" ::"r"(ptx::smem_u32(at)), "r"(lo.x), "r"(lo.y), "r"(lo.z), "r"(lo.w) : "memory");
            asm volatile("st.shared.v4.u32 [%0], {%1,%2,%3,%4};" ::"r"(ptx::smem_u32(at + 16)), "r"(hi.x), "r"(hi.y), "r"(hi.z), "r"(hi.w) : "memory");
          }
        } else if (d.flags & kAuxInSlot) {
          // one destination: the producer brought the second operand's tile along with the sources
          const uint4 rq = lds16(slot + (size_t)(ns + __popc(pmask)) * tile + (size_t)u * 16u);
          const bool f32 = (DT == PL_BF16) && (P.hook & PL_HOOK_F32_OUT);
          store_final_q<DT>(acc, P.out_scale, P.hook, static_cast<char*>(P.base[d.dst_slot]) + d.dst_off + (size_t)u * (f32 ? 32u : 16u), rq);
        } else {
          store_final_unit<DT>(P, acc, d.dst_slot, d.dst_off, bcast, u);
        }
      }
    } else if (dpart) {
      if constexpr (DT == PL_BF16) {
        st16(d.dst + (size_t)u * 32u, make_uint4(__float_as_uint(acc.v[0]), __float_as_uint(acc.v[1]),
                                                  __float_as_uint(acc.v[2]), __float_as_uint(acc.v[3])));
        st16(d.dst + (size_t)u * 32u + 16u, make_uint4(__float_as_uint(acc.v[4]), __float_as_uint(acc.v[5]),
                                                        __float_as_uint(acc.v[6]), __float_as_uint(acc.v[7])));
      } else if constexpr (DT == PL_F32) {
        st16(d.dst + (size_t)u * 32u, acc.sums());
        st16(d.dst + (size_t)u * 32u + 16u, acc.corrections());
      }
    } else {
      uint4 r;
      if constexpr (DT == PL_BF16) r = acc.to_bf16(P.out_scale);
      else r = acc.result(P.out_scale);
      if (!bcast) {
        st16(d.dst + (size_t)u * 16u, r);
      } else if (pmask == 0) {
        // Replicated destination: park the result in the slot, over unit u of the first source
        // tile (this thread has already read unit u of every tile and nobody else reads it);
        // the copier sends the tile to all R outputs with bulk stores.
        asm volatile("st.shared.v4.u32 [%0], {%1,%2,%3,%4};" ::"r"(ptx::smem_u32(slot + (size_t)u * 16u)), "r"(r.x),
                     "r"(r.y), "r"(r.z), "r"(r.w)
                     : "memory");
      } else {
        for (int k = 0; k < P.n_ranks; ++k)
          st16(static_cast<char*>(P.base[kSlotOut + k]) + d.dst_off + (size_t)u * 16u, r);
      }
    }
  }
  if ((bcast && pmask == 0 && !final_op) || (HOOK && (d.flags & kResInSlot))) ptx::fence_proxy_async_smem();  // generic writes above -> the copier's bulk stores
}

// ---- software-pipelined path for plain reduce stages ---------------------------------------
// A stage is "plain" when every source is element-typed, there are at most 8 of them, the
// result goes to one element-typed destination and the stage does not publish a flag: the
// whole of a direct reduce-scatter.  For such stages a consumer thread owns exactly one
// 16-byte unit per trip; it pulls its operands into registers and hands the slot back to the
// producer at once, and it does so for stage n+1 BEFORE it runs the adds and the store of
// stage n whenever stage n+1 has already landed.  A landed slot then waits for one round of
// shared-memory loads instead of a whole stage of arithmetic (measured on B200, reduce-scatter
// of 8 x 64 MiB: the ring held ~1.5 of its 4 slots for the consumers, which kept the bytes in
// flight below what saturates HBM).
struct PlainStage {
  char* dst;        // destination of the stage's unit 0
  uint32_t units;   // units in the stage
  uint32_t ns;      // sources
  bool dpart;       // destination holds partials (twice as wide)
};

// A thread keeps 8 operand vectors of a stage: 1 unit of up to 8 sources, 2 units of up to 4
// or 4 units of up to 2, unit j of thread t being unit t + j * (32 * CW) of the stage.  The producer sizes plain stages of
// the pipelined variant accordingly (plain_unit_cap).
__device__ __forceinline__ uint32_t plain_units_per_thread(uint32_t ns) { return ns > 4 ? 1u : ns > 2 ? 2u : 4u; }
template <int CW>
__device__ __forceinline__ uint32_t plain_unit_cap(uint32_t ns) { return (uint32_t)(32 * CW) * plain_units_per_thread(ns); }

template <int CW>
__device__ __forceinline__ bool stage_is_plain(const StageDesc& d) {
  return d.kind != PL_OP_COPY && d.kind != kEnd && d.pmask == 0 && d.n_src >= 1 && d.n_src <= 8 && !(d.flags & kDstBcast) &&
         !((d.flags & kLastOfOp) && d.signal != kNoFlag) && d.units <= plain_unit_cap<CW>(d.n_src);
}

// Operands of this thread's units into q[]: NSMAX (8, 4 or 2) bounds the source count, so the
// register index of every operand is a compile-time constant.
template <int CW, int NSMAX>
__device__ __forceinline__ void plain_load_ns(const unsigned char* slot, uint32_t tile, uint32_t units, uint32_t ns, int ctid,
                                              uint4 (&q)[8]) {
  constexpr int UPT = 8 / NSMAX;
#pragma unroll
  for (int j = 0; j < UPT; ++j) {
    const uint32_t u = (uint32_t)ctid + (uint32_t)(j * 32 * CW);
    if (u < units) {
#pragma unroll
      for (int k = 0; k < NSMAX; ++k)
        if ((uint32_t)k < ns) q[j * NSMAX + k] = lds16(slot + (size_t)k * tile + (size_t)u * 16u);
    }
  }
}

// Descriptor fields into st, operands into q[], slot released.
template <int CW>
__device__ __forceinline__ void plain_load(const StageDesc& d, const unsigned char* slot, int ctid, uint64_t* empty,
                                           PlainStage& st, uint4 (&q)[8]) {
  st.units = d.units;
  st.ns = d.n_src;
  st.dpart = d.flags & kDstF32;
  st.dst = d.dst;
  const uint32_t tile = d.ucap * 16u;
  if (st.ns > 4) plain_load_ns<CW, 8>(slot, tile, st.units, st.ns, ctid, q);
  else if (st.ns > 2) plain_load_ns<CW, 4>(slot, tile, st.units, st.ns, ctid, q);
  else plain_load_ns<CW, 2>(slot, tile, st.units, st.ns, ctid, q);
  __syncwarp();
  // the arrive is a release: this warp's shared-memory loads above are performed before it
  if ((ctid & 31) == 0) ptx::mbar_arrive(empty);
}

template <int DT, int CW, int NSMAX>
__device__ __forceinline__ void plain_finish_ns(const ExecParams& P, const PlainStage& st, const uint4 (&q)[8], int ctid) {
  constexpr int UPT = 8 / NSMAX;
#pragma unroll
  for (int j = 0; j < UPT; ++j) {
    const uint32_t u = (uint32_t)ctid + (uint32_t)(j * 32 * CW);
    if (u >= st.units) continue;
    Acc<DT> acc;
    acc.zero();
#pragma unroll
    for (int k = 0; k < NSMAX; ++k)
      if ((uint32_t)k < st.ns) {
        if constexpr (DT == PL_BF16) acc.add_bf16(q[j * NSMAX + k]);
        else acc.add(q[j * NSMAX + k]);
      }
    if (st.dpart) {
      if constexpr (DT == PL_BF16) {
        st16(st.dst + (size_t)u * 32u, make_uint4(__float_as_uint(acc.v[0]), __float_as_uint(acc.v[1]),
                                                  __float_as_uint(acc.v[2]), __float_as_uint(acc.v[3])));
        st16(st.dst + (size_t)u * 32u + 16u, make_uint4(__float_as_uint(acc.v[4]), __float_as_uint(acc.v[5]),
                                                        __float_as_uint(acc.v[6]), __float_as_uint(acc.v[7])));
      } else if constexpr (DT == PL_F32) {
        st16(st.dst + (size_t)u * 32u, acc.sums());
        st16(st.dst + (size_t)u * 32u + 16u, acc.corrections());
      }
    } else {
      uint4 r;
      if constexpr (DT == PL_BF16) r = acc.to_bf16(P.out_scale);
      else r = acc.result(P.out_scale);
      st16(st.dst + (size_t)u * 16u, r);
    }
  }
}

template <int DT, int CW>
__device__ __forceinline__ void plain_finish(const ExecParams& P, const PlainStage& st, const uint4 (&q)[8], int ctid) {
  if (st.ns > 4) plain_finish_ns<DT, CW, 8>(P, st, q, ctid);
  else if (st.ns > 2) plain_finish_ns<DT, CW, 4>(P, st, q, ctid);
  else plain_finish_ns<DT, CW, 2>(P, st, q, ctid);
}

// A REDUCE stage whose result leaves through shared memory (see consume_stage).
template <bool HOOK>
__device__ __forceinline__ bool leaves_via_smem(uint32_t kind, uint32_t flags, uint32_t pmask) {
  if (kind == PL_OP_COPY) return false;
  if (HOOK && (flags & kResInSlot)) return true;
  return (flags & kDstBcast) && !(flags & (kDstF32 | kFinal)) && pmask == 0;
}

// HOOK: the variant for schedules with a processing phase beyond the scale (general consumers only).
// DBUF: the variant for staged schedules with two staging buffers (PL_OPT_STAGE_AHEAD): flag set
// and staging buffer follow the parity of a launch counter taken at entry; the producer runs the
// leading stage ops of its queue (copies from the caller's input into the staging buffer of this
// parity) before it waits for the launch in front, the copier ships them, the consumers wait.
// SM-window launches (write-dominated schedules without flags): see window_claim in pl_device.cuh.
__device__ __forceinline__ int claim_queue(const ExecParams& P) {
  bool timed_out = false;
  const int q = window_claim(P.sm_state, P.sm_mask, P.n_queues, 2ull * P.timeout_ns + 1000000ull, &timed_out);
  // CTAs of this launch still missing after the time limit: queues may go unclaimed, say so
  if (timed_out) record_timeout(P, (int)blockIdx.x, 0xFFFFFFFFu, 0xFFFFFFFFu, gridDim.x, 0);
  return q;
}
__device__ __forceinline__ void leave_window(const ExecParams& P) { window_leave(P.sm_state); }

template <int DT, int CW, bool HOOK = false, bool DBUF = false>
__global__ void __launch_bounds__(32 * (kProducers + 1 + CW), 1) pl_exec_tma_kernel(const __grid_constant__ ExecParams P) {
  extern __shared__ __align__(1024) unsigned char smem[];
  Ctrl* c = reinterpret_cast<Ctrl*>(smem);
  unsigned char* slots = smem + kCtrlBytes;
  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  int q = blockIdx.x;
  uint32_t n_cta = gridDim.x;  // CTAs that work in this launch
  if constexpr (!DBUF) {
    if (P.sm_state != nullptr) {
      if (tid == 0) c->q = claim_queue(P);
      __syncthreads();
      q = c->q;
      n_cta = P.n_queues;
      if (q < 0) {  // this SM sits the launch out (an exited CTA counts as having let dependents go)
        if (tid == 0) leave_window(P);
        return;
      }
    }
  }
  const uint32_t S = (uint32_t)P.stages, slot_bytes = P.stage_bytes;
  const bool has_flags = P.flags != nullptr;
  if constexpr (!DBUF) pdl_launch_dependents();

  if (tid == 0) {
    if constexpr (DBUF) c->launch = atomicAdd(P.epoch + 2, 1ull) / gridDim.x;  // ticket: see the register executor
    for (uint32_t s = 0; s < S; ++s) {
      ptx::mbar_init(&c->full[s], 1);
      ptx::mbar_init(&c->empty[s], 1 + CW);  // copier + every consumer warp
    }
    for (uint32_t s = 0; s < S; ++s) ptx::mbar_init(&c->done[s], CW);
    c->abort = 0;
    c->q = q;
    ptx::mbar_init_fence();
  }
  // Producers: the first descriptor of the queue.  Descriptors are written when the schedule is
  // built and never by a kernel, so this load may run ahead of the wait for the launch in front.
  const uint32_t nq = P.n_queues;
  uint4 r_op = make_uint4(0, 0, 0, 0), r_op_next = r_op;
  uint64_t r_src = 0, r_src_next = 0;
  DevWait r_wait = {0, 0}, r_wait_next = {0, 0};
  auto fetch = [&](uint32_t i, uint4& o, uint64_t& sr, DevWait& w) {
    const uint64_t at = (uint64_t)i * nq + q;  // op i of this queue
    if (lane < 4) o = reinterpret_cast<const uint4*>(P.ops + at)[lane];
    if (lane < (int)P.src_stride) sr = P.srcs[at * P.src_stride + lane];
    if (lane < (int)P.wait_stride) w = P.waits[at * P.wait_stride + lane];
  };
  if (warp < kProducers) fetch(0, r_op_next, r_src_next, r_wait_next);

  unsigned long long epoch = 0ull, scratch_shift = 0ull;
  unsigned long long* flag_base = P.flags;
  if constexpr (DBUF) {
    __syncthreads();
    const unsigned long long launch = c->launch;
    epoch = (launch >> 1) + 1ull;
    if (launch & 1ull) {
      scratch_shift = P.scratch_half;
      flag_base = P.flags + P.n_flags;
    }
    // consumers only ever handle reduce stages, which come after the producer's wait: they may
    // block here; the producer waits later (below), the copier not at all (it reads shared
    // memory only, and what it stores or signals belongs to this launch's own buffer and flag set
    // until the producer has waited)
    if (warp > kProducers) pdl_wait();
  } else {
    pdl_wait();  // from here on memory written by earlier launches may be read
    epoch = has_flags ? *reinterpret_cast<volatile unsigned long long*>(P.epoch) + 1ull : 0ull;
    __syncthreads();
  }

  if (warp < kProducers) {
    // ================================ producers ========================================
    // Both walk the whole queue (descriptors, flag waits, stage arithmetic); a stage is filled
    // by the producer whose number equals the stage number modulo kProducers.
    uint32_t n = 0;  // stages produced
    bool ok = true;
    // the first descriptor tells how many ops the queue holds (a placeholder marks an empty one)
    const uint32_t first_kind = __shfl_sync(0xFFFFFFFFu, r_op_next.x, 0);
    const uint32_t n_ops = first_kind == kNopKind ? 0u : __shfl_sync(0xFFFFFFFFu, r_op_next.z, 0) + 1u;
    bool waited = !DBUF;
    for (uint32_t i = 0; i < n_ops && ok; ++i) {
      r_op = r_op_next;
      r_src = r_src_next;
      r_wait = r_wait_next;
      if (i + 1 < n_ops) fetch(i + 1, r_op_next, r_src_next, r_wait_next);
      if constexpr (DBUF) {
        // the first op that is not an early stage op: wait for the launch in front, then let the
        // launch behind start (it will write the staging buffer this launch's predecessor used)
        if (!waited && !(__shfl_sync(0xFFFFFFFFu, r_op.w, 1) & kStageAhead)) {
          pdl_wait();
          pdl_launch_dependents();
          waited = true;
        }
      }
      // op words: lane 0: kind n_src remaining pmask | lane 1: rsv n_wait signal flags | lane 2: count dst | lane 3: topo signal2
      const uint32_t kind = __shfl_sync(0xFFFFFFFFu, r_op.x, 0), n_src = __shfl_sync(0xFFFFFFFFu, r_op.y, 0);
      const uint32_t pmask = __shfl_sync(0xFFFFFFFFu, r_op.w, 0);
      const uint32_t n_wait = __shfl_sync(0xFFFFFFFFu, r_op.y, 1), signal = __shfl_sync(0xFFFFFFFFu, r_op.z, 1);
      const uint32_t oflags = __shfl_sync(0xFFFFFFFFu, r_op.w, 1);
      const uint64_t count = ((uint64_t)__shfl_sync(0xFFFFFFFFu, r_op.y, 2) << 32) | __shfl_sync(0xFFFFFFFFu, r_op.x, 2);
      const uint64_t dstp = ((uint64_t)__shfl_sync(0xFFFFFFFFu, r_op.w, 2) << 32) | __shfl_sync(0xFFFFFFFFu, r_op.z, 2);
      const uint32_t topo = __shfl_sync(0xFFFFFFFFu, r_op.x, 3), signal2 = __shfl_sync(0xFFFFFFFFu, r_op.y, 3);

      // ---- wait (acquire) on the op's flags: lane k polls entry k
      bool lane_ok = true;
      if (lane < (int)n_wait) {
        const unsigned long long need = epoch * (unsigned long long)r_wait.need;
        const unsigned long long* fp = flag_base + r_wait.flag;
        unsigned long long seen = ld_acquire_u64(fp);
        if (seen < need) {
          const unsigned long long t0 = globaltimer_ns();
          uint32_t spins = 0;
          while ((seen = ld_acquire_u64(fp)) < need) {
            if ((++spins & 63u) == 0) {
              if (ld_volatile_s32(P.status + 8) || *reinterpret_cast<volatile int*>(&c->abort)) { lane_ok = false; break; }
              if (globaltimer_ns() - t0 > P.timeout_ns) {
                record_timeout(P, q, topo, r_wait.flag, need, seen);
                lane_ok = false;
                break;
              }
            }
          }
        }
      }
      ok = __all_sync(0xFFFFFFFFu, lane_ok);
      if (!ok) break;
      if (n_wait) ptx::fence_proxy_async();  // data released by other CTAs' generic stores -> our bulk loads
      if (P.trace && tid == 0) P.trace[2ull * topo] = globaltimer_ns();  // waits satisfied

      // ---- cut the op into stages
      const char* my_src = (lane < (int)n_src) ? (DBUF ? resolve(P, r_src, scratch_shift) : resolve(P, r_src)) : nullptr;
      const bool my_part = (pmask >> lane) & 1u;
      // Final op of a schedule with a second operand and one destination: that operand's tile
      // rides in the slot behind the sources (one more bulk load per stage), so that no consumer
      // waits for a global load with the slot in its hands.
      bool aux_tile = false;
      if constexpr (HOOK) aux_tile = kind != PL_OP_COPY && (oflags & kFinal) && !(oflags & kDstBcast) && (P.hook & PL_HOOK_RESIDUAL);
      // Final op with R destinations: results leave through the slot (kResInSlot) when the slot
      // can hold them: a second operand per rank and element-typed output (R operand tiles,
      // overwritten in place by the R results), or fp32 output without a second operand (one
      // result region of 32 bytes per unit).  Both at once would leave too few units per stage:
      // those schedules keep the consumers' per-destination global stores.
      uint32_t res_mode = 0;  // 1: per-rank results over the operand tiles, 2: one wide result region
      if constexpr (HOOK) {
        if (kind != PL_OP_COPY && (oflags & kFinal) && (oflags & kDstBcast) && pmask == 0) {
          const bool residual = P.hook & PL_HOOK_RESIDUAL, wide = (DT == PL_BF16) && (P.hook & PL_HOOK_F32_OUT);
          if (residual && !wide && n_src + (uint32_t)P.n_ranks <= 32u) res_mode = 1;
          else if (!residual && wide) res_mode = 2;
        }
      }
      const uint32_t extra_b = aux_tile ? 16u : res_mode == 1 ? 16u * (uint32_t)P.n_ranks : res_mode == 2 ? 32u : 0u;
      const uint32_t unit_b = (kind == PL_OP_COPY) ? 16u : 16u * (n_src + __popc(pmask)) + extra_b;  // slot bytes per unit
      const uint32_t load_b = unit_b - (res_mode == 2 ? 32u : 0u);  // of which the bulk loads fill (a result region is not loaded)
      uint32_t ucap = slot_bytes / unit_b;
      if constexpr (CW == kWarpsPipelined) {
        // plain reduce op: a stage holds what the consumer threads can keep in registers
        if (kind != PL_OP_COPY && pmask == 0 && n_src >= 1 && n_src <= 8 && !(oflags & kDstBcast))
          ucap = min(ucap, plain_unit_cap<CW>(n_src));
      }
      const uint64_t n_units = (kind == PL_OP_COPY) ? (count >> 4) : count / Acc<DT == PL_U8 ? PL_I32 : DT>::kElems;
      // tile offset of my source inside a slot, and my bytes per unit
      const uint32_t my_w = my_part ? 32u : 16u;
      const uint32_t my_tile_off = ucap * 16u * (lane + __popc(pmask & ((1u << lane) - 1u)));
      const uint32_t dst_w = (kind == PL_OP_COPY) ? 16u : ((oflags & kDstF32) ? 32u : 16u);
      char* dst = DBUF ? resolve(P, dstp, scratch_shift) : resolve(P, dstp);
      const uint64_t dst_off = dstp & 0xFFFFFFFFFFFFull;
      const char* aux_src = nullptr;
      if (aux_tile) {
        const bool f32 = (DT == PL_BF16) && (P.hook & PL_HOOK_F32_OUT);  // the output is twice as wide as the operand
        aux_src = static_cast<const char*>(P.base[kSlotAux + ((dstp >> 48) - kSlotOut)]) + (f32 ? dst_off >> 1 : dst_off);
      }
      const uint32_t aux_tile_off = HOOK ? ucap * 16u * (n_src + __popc(pmask)) : 0u;
      for (uint64_t u0 = 0; u0 < n_units; u0 += ucap) {
        if (n % kProducers != (uint32_t)warp) {  // the other producer's stage
          ++n;
          continue;
        }
        const uint32_t units = (uint32_t)min((uint64_t)ucap, n_units - u0);
        const uint32_t s = n % S, ph = (n / S) & 1u;
        bool w_ok = true;
        if (lane == 0) w_ok = wait_bar(P, c, &c->empty[s], ph ^ 1u);
        ok = __shfl_sync(0xFFFFFFFFu, (int)w_ok, 0);
        if (!ok) break;
        if (lane == 0) {
          StageDesc& d = c->desc[s];
          d.kind = kind;
          d.n_src = n_src;
          d.units = units;
          d.ucap = ucap;
          d.pmask = pmask;
          d.flags = oflags | ((u0 + ucap >= n_units) ? kLastOfOp : 0u) | (aux_tile ? kAuxInSlot : 0u) | (res_mode ? kResInSlot : 0u);
          // signals go to this launch's flag set
          d.signal = (DBUF && signal != kNoFlag && flag_base != P.flags) ? signal + P.n_flags : signal;
          d.signal2 = (DBUF && signal2 != kNoFlag && flag_base != P.flags) ? signal2 + P.n_flags : signal2;
          d.dst = dst + u0 * dst_w;
          d.dst_off = dst_off + u0 * dst_w;
          d.topo = topo;
          d.dst_slot = (uint32_t)(dstp >> 48);
          ptx::mbar_expect_tx(&c->full[s], units * load_b);
        }
        __syncwarp();
        if (lane < (int)n_src) {
          void* sdst = slots + (size_t)s * slot_bytes + my_tile_off;
          if ((P.hints & 4u) && kind == PL_OP_COPY && !(oflags & kDstBcast)) ptx::bulk_g2s_hint(sdst, my_src + u0 * my_w, units * my_w, &c->full[s], ptx::policy_evict_last());
          else if ((P.hints & 1u) && (r_src >> 48) < (uint64_t)kSlotOut) ptx::bulk_g2s_hint(sdst, my_src + u0 * my_w, units * my_w, &c->full[s], ptx::policy_evict_first());
          else ptx::bulk_g2s(sdst, my_src + u0 * my_w, units * my_w, &c->full[s]);
        }
        if (aux_tile && lane == (int)n_src)
          ptx::bulk_g2s(slots + (size_t)s * slot_bytes + aux_tile_off, aux_src + u0 * 16u, units * 16u, &c->full[s]);
        if (res_mode == 1 && lane >= (int)n_src && lane < (int)n_src + P.n_ranks) {
          // rank k's second operand for this stage (laid out like the element-typed output)
          const int k = lane - (int)n_src;
          ptx::bulk_g2s(slots + (size_t)s * slot_bytes + aux_tile_off + (size_t)k * ucap * 16u,
                        static_cast<const char*>(P.base[kSlotAux + k]) + dst_off + u0 * 16u, units * 16u, &c->full[s]);
        }
        ++n;
      }
    }
    if constexpr (DBUF) {
      if (!waited) {  // a queue of early stage ops only (or an empty one)
        pdl_wait();
        pdl_launch_dependents();
      }
    }
    // ---- end of queue (or abort): tell the other warps, then make sure nothing is in flight
    if (lane == 0) {
      if (!ok) {
        *reinterpret_cast<volatile int*>(&c->abort) = 1;
        // loads this warp issued must land before the CTA may leave: bounded drain
        for (uint32_t k = (n > S ? n - S : 0u); k < n; ++k)
          if (k % kProducers == (uint32_t)warp)
            for (uint32_t tries = 0; tries < (1u << 22) && !ptx::mbar_try_wait(&c->full[k % S], (k / S) & 1u); ++tries) {}
      }
      // the end marker is the stage after the last one: it belongs to one of the producers too
      const uint32_t s = n % S, ph = (n / S) & 1u;
      if (ok && n % kProducers == (uint32_t)warp && wait_bar(P, c, &c->empty[s], ph ^ 1u)) {
        c->desc[s].kind = kEnd;
        ptx::mbar_arrive(&c->full[s]);
      }
    }
  } else if (warp == kProducers) {
    // ================================ copier ============================================
    int prev = -1;  // slot whose bulk store may still be reading shared memory
    uint32_t done_parity = 0;  // tracked exactly as the consumers do
    for (uint32_t n = 0;; ++n) {
      const uint32_t s = n % S, ph = (n / S) & 1u;
      bool go = true;
      if (lane == 0) go = wait_bar(P, c, &c->full[s], ph);
      go = __shfl_sync(0xFFFFFFFFu, (int)go, 0);
      __syncwarp();  // lane 0's acquire on the barrier covers the whole warp's reads below
      if (!go) break;
      const StageDesc& d = c->desc[s];
      const uint32_t kind = d.kind;
      if (kind == kEnd) break;
      const bool via_smem = leaves_via_smem<HOOK>(kind, d.flags, d.pmask);
      const bool to_all = via_smem || (kind == PL_OP_COPY && (d.flags & kDstBcast));  // one tile, R destinations
      const bool uses_done = via_smem || (kind != PL_OP_COPY && (d.flags & kLastOfOp) && d.signal != kNoFlag);
      if (via_smem) {
        bool ready = true;
        if (lane == 0) ready = wait_bar(P, c, &c->done[s], (done_parity >> s) & 1u);  // all consumer warps wrote
        ready = __shfl_sync(0xFFFFFFFFu, (int)ready, 0);
        if (!ready) break;
      }
      if (uses_done) done_parity ^= 1u << s;
      if (lane == 0) {
        if (kind == PL_OP_COPY || via_smem) {
          if (to_all) {
            const bool res = HOOK && (d.flags & kResInSlot);
            const uint32_t stride = res ? res_stride(P, d) : 0u;
            const uint32_t bytes = d.units * ((res && !stride) ? 32u : 16u);
            for (int k = 0; k < P.n_ranks; ++k) {
              void* dk = static_cast<char*>(P.base[kSlotOut + k]) + d.dst_off;
              const unsigned char* from = slots + (size_t)s * slot_bytes + (res ? res_off(d) + (size_t)k * stride : 0u);
              if (P.hints & 2u) ptx::bulk_s2g_hint(dk, from, bytes, ptx::policy_evict_first());
              else ptx::bulk_s2g(dk, from, bytes);
            }
          } else if (P.hints & 2u) {
            ptx::bulk_s2g_hint(d.dst, slots + (size_t)s * slot_bytes, d.units * 16u, ptx::policy_evict_first());
          } else {
            ptx::bulk_s2g(d.dst, slots + (size_t)s * slot_bytes, d.units * 16u);
          }
          ptx::bulk_commit();
          if (prev >= 0) {
            ptx::bulk_wait_read<1>();
            ptx::mbar_arrive(&c->empty[prev]);
          }
          prev = (int)s;
          if ((d.flags & kLastOfOp) && d.signal != kNoFlag) {
            ptx::bulk_wait<0>();        // the op's bytes have landed
            ptx::fence_proxy_async();   // async-proxy writes before the generic-proxy release
            if (P.trace) P.trace[2ull * d.topo + 1] = globaltimer_ns();
            __threadfence();
            red_release_add_u64(P.flags + d.signal, 1ull);
            if (d.signal2 != kNoFlag) red_release_add_u64(P.flags + d.signal2, 1ull);
          }
        } else {
          if (prev >= 0) {
            ptx::bulk_wait_read<0>();
            ptx::mbar_arrive(&c->empty[prev]);
            prev = -1;
          }
          ptx::mbar_arrive(&c->empty[s]);
        }
      }
    }
    if (lane == 0) {
      ptx::bulk_wait<0>();
      if (prev >= 0) ptx::mbar_arrive(&c->empty[prev]);
    }
  } else {
    // ================================ consumers =========================================
    const int ctid = tid - 32 * (kProducers + 1);
    uint32_t done_parity = 0;  // bit s: parity of the next phase of done[s]
    // operands of a plain stage that were pulled into registers ahead of time
    bool have = false;
    PlainStage st_a = {nullptr, 0u, 0u, false};
    uint4 q_a[8];
    for (uint32_t n = 0;; ++n) {
      const uint32_t s = n % S, ph = (n / S) & 1u;
      if constexpr (DT != PL_U8 && CW == kWarpsPipelined) {
        if (have) {
          // Stage n-1 sits in registers and its slot is already back with the producer.  If
          // stage n has landed and is plain too, take its operands first, then finish n-1.
          bool next = false;
          if (lane == 0) next = ptx::mbar_try_wait(&c->full[s], ph);
          next = __shfl_sync(0xFFFFFFFFu, (int)next, 0);
          __syncwarp();  // lane 0's acquire on the barrier covers the whole warp's reads below
          if (next) next = stage_is_plain<CW>(c->desc[s]);
          if (next) {
            PlainStage st_b;
            uint4 q_b[8];
            plain_load<CW>(c->desc[s], slots + (size_t)s * slot_bytes, ctid, &c->empty[s], st_b, q_b);
            plain_finish<DT, CW>(P, st_a, q_a, ctid);
            st_a = st_b;
#pragma unroll
            for (int k = 0; k < 8; ++k) q_a[k] = q_b[k];
            continue;
          }
          plain_finish<DT, CW>(P, st_a, q_a, ctid);
          have = false;  // stage n is handled below
        }
      }
      bool go = true;
      if (lane == 0) go = wait_bar(P, c, &c->full[s], ph);
      go = __shfl_sync(0xFFFFFFFFu, (int)go, 0);
      __syncwarp();  // lane 0's acquire on the barrier covers the whole warp's reads below
      if (!go) break;
      const StageDesc& d = c->desc[s];
      const uint32_t kind = d.kind;
      if (kind == kEnd) break;
      if constexpr (DT != PL_U8 && CW == kWarpsPipelined) {
        if (stage_is_plain<CW>(d)) {
          plain_load<CW>(d, slots + (size_t)s * slot_bytes, ctid, &c->empty[s], st_a, q_a);
          have = true;
          continue;
        }
      }
      if (kind != PL_OP_COPY) {
        if constexpr (DT != PL_U8) consume_stage<DT, CW, HOOK>(P, d, slots + (size_t)s * slot_bytes, ctid);
        const bool last = d.flags & kLastOfOp;
        const uint32_t signal = d.signal, signal2 = d.signal2, topo = d.topo;
        __syncwarp();
        if (leaves_via_smem<HOOK>(kind, d.flags, d.pmask)) {
          // the copier ships the tile (and signals, if this is the op's last stage)
          if (lane == 0) ptx::mbar_arrive(&c->done[s]);
          done_parity ^= 1u << s;
        } else if (last && signal != kNoFlag) {
          // every consumer warp reports its stores; consumer thread 0 then publishes
          if (lane == 0) ptx::mbar_arrive(&c->done[s]);
          if (ctid == 0) {
            if (wait_bar(P, c, &c->done[s], (done_parity >> s) & 1u)) {
              if (P.trace) P.trace[2ull * topo + 1] = globaltimer_ns();
              __threadfence();
              red_release_add_u64(P.flags + signal, 1ull);
              if (signal2 != kNoFlag) red_release_add_u64(P.flags + signal2, 1ull);
            }
          }
          done_parity ^= 1u << s;
        }
      }
      __syncwarp();
      if (lane == 0) ptx::mbar_arrive(&c->empty[s]);
    }
  }

  __syncthreads();
  if constexpr (!DBUF) {
    if (tid == 0 && P.sm_state != nullptr) leave_window(P);
  }
  if (tid == 0 && has_flags && !DBUF && !*reinterpret_cast<volatile int*>(&c->abort)) {
    const unsigned long long prev = atomicAdd(P.epoch + 1, 1ull);
    if (prev == (unsigned long long)n_cta - 1ull) {
      P.epoch[1] = 0ull;
      __threadfence();
      *reinterpret_cast<volatile unsigned long long*>(P.epoch) = epoch;
    }
  }
}

template <int DT, int CW, bool HOOK = false, bool DBUF = false>
cudaError_t launch_t(const ExecParams& P, int grid, cudaStream_t stream) {
  const size_t smem = exec_tma_smem_bytes(P.stages, P.stage_bytes);
  // the shared-memory opt-in is a per-device attribute of the function: one bit per device
  static std::atomic<unsigned long long> configured{0};  // per instantiation
  int dev = 0;
  cudaError_t e = cudaGetDevice(&dev);
  if (e != cudaSuccess) return e;
  const unsigned long long bit = 1ull << (dev & 63);
  if (!(configured.load(std::memory_order_acquire) & bit)) {
    e = cudaFuncSetAttribute(pl_exec_tma_kernel<DT, CW, HOOK, DBUF>, cudaFuncAttributeMaxDynamicSharedMemorySize, 227 * 1024);
    if (e != cudaSuccess) return e;
    configured.fetch_or(bit, std::memory_order_release);
  }
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = dim3((unsigned)grid);
  cfg.blockDim = dim3((unsigned)(32 * (kProducers + 1 + CW)));
  cfg.dynamicSmemBytes = smem;
  cfg.stream = stream;
  cudaLaunchAttribute attr[1];
  attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  attr[0].val.programmaticStreamSerializationAllowed = 1;
  cfg.attrs = attr;
  cfg.numAttrs = P.overlap_launch ? 1 : 0;
  return cudaLaunchKernelEx(&cfg, pl_exec_tma_kernel<DT, CW, HOOK, DBUF>, P);
}

template <int DT, int CW, bool HOOK = false, bool DBUF = false>
int occupancy_t(size_t smem) {
  int n = 0;
  if (cudaFuncSetAttribute(pl_exec_tma_kernel<DT, CW, HOOK, DBUF>, cudaFuncAttributeMaxDynamicSharedMemorySize, 227 * 1024) != cudaSuccess ||
      cudaOccupancyMaxActiveBlocksPerMultiprocessor(&n, pl_exec_tma_kernel<DT, CW, HOOK, DBUF>, 32 * (kProducers + 1 + CW), smem) != cudaSuccess) {
    cudaGetLastError();
    return 0;
  }
  return n;
}

}  // namespace

size_t exec_tma_smem_bytes(int stages, uint32_t stage_bytes) { return kCtrlBytes + (size_t)stages * stage_bytes; }
int exec_tma_threads(bool pipelined) { return 32 * (kProducers + 1 + (pipelined ? kWarpsPipelined : kWarpsGeneral)); }

cudaError_t launch_exec_tma(int dtype, const ExecParams& P, int grid, cudaStream_t stream) {
  if (P.stages < 2 || P.stages > kMaxStages) return cudaErrorInvalidValue;
  if (P.stage_ahead) {
    switch (dtype) {
      case PL_BF16: return launch_t<PL_BF16, kWarpsGeneral, false, true>(P, grid, stream);
      case PL_F32: return launch_t<PL_F32, kWarpsGeneral, false, true>(P, grid, stream);
      case PL_I32: return launch_t<PL_I32, kWarpsGeneral, false, true>(P, grid, stream);
      default: return launch_t<PL_U8, kWarpsGeneral, false, true>(P, grid, stream);
    }
  }
  if (P.hook) {
    switch (dtype) {
      case PL_BF16: return launch_t<PL_BF16, kWarpsGeneral, true>(P, grid, stream);
      case PL_F32: return launch_t<PL_F32, kWarpsGeneral, true>(P, grid, stream);
      default: return cudaErrorInvalidValue;
    }
  }
  if (P.pipelined_reduce) {
    switch (dtype) {
      case PL_BF16: return launch_t<PL_BF16, kWarpsPipelined>(P, grid, stream);
      case PL_F32: return launch_t<PL_F32, kWarpsPipelined>(P, grid, stream);
      case PL_I32: return launch_t<PL_I32, kWarpsPipelined>(P, grid, stream);
      default: break;  // byte schedules have no reduce stages
    }
  }
  switch (dtype) {
    case PL_BF16: return launch_t<PL_BF16, kWarpsGeneral>(P, grid, stream);
    case PL_F32: return launch_t<PL_F32, kWarpsGeneral>(P, grid, stream);
    case PL_I32: return launch_t<PL_I32, kWarpsGeneral>(P, grid, stream);
    default: return launch_t<PL_U8, kWarpsGeneral>(P, grid, stream);
  }
}

// resident CTAs per SM that hold for either variant of the kernel
int exec_tma_max_ctas_per_sm(int dtype, int stages, uint32_t stage_bytes) {
  const size_t smem = exec_tma_smem_bytes(stages, stage_bytes);
  if (smem > 227 * 1024) return 0;
  switch (dtype) {
    case PL_BF16: return std::min({occupancy_t<PL_BF16, kWarpsGeneral>(smem), occupancy_t<PL_BF16, kWarpsPipelined>(smem),
                                   occupancy_t<PL_BF16, kWarpsGeneral, true>(smem), occupancy_t<PL_BF16, kWarpsGeneral, false, true>(smem)});
    case PL_F32: return std::min({occupancy_t<PL_F32, kWarpsGeneral>(smem), occupancy_t<PL_F32, kWarpsPipelined>(smem),
                                  occupancy_t<PL_F32, kWarpsGeneral, true>(smem), occupancy_t<PL_F32, kWarpsGeneral, false, true>(smem)});
    case PL_I32: return std::min({occupancy_t<PL_I32, kWarpsGeneral>(smem), occupancy_t<PL_I32, kWarpsPipelined>(smem),
                                  occupancy_t<PL_I32, kWarpsGeneral, false, true>(smem)});
    default: return std::min(occupancy_t<PL_U8, kWarpsGeneral>(smem), occupancy_t<PL_U8, kWarpsGeneral, false, true>(smem));
  }
}

}  // namespace pl
