// Device-side helpers shared by the executor kernels: flag accesses with acquire / release
// semantics, 128-bit global accesses, the per-dtype accumulators (Sec. 3.3, Eq. "rank-order":
// convert to fp32, one accumulator per element, ascending source order, convert once), and
// the time-out record.
#pragma once
#include <cuda_bf16.h>
#include <cuda_runtime.h>

#include "pl_internal.h"

namespace pl {
namespace dev {

// ---- small PTX helpers ---------------------------------------------------------------
__device__ __forceinline__ unsigned long long ld_acquire_u64(const unsigned long long* p) {
  unsigned long long v;
  asm volatile("ld.acquire.gpu.global.u64 %0, [%1];" : "=l"(v) : "l"(p) : "memory");
  return v;
}
__device__ __forceinline__ void red_release_add_u64(unsigned long long* p, unsigned long long v) {
  asm volatile("red.release.gpu.global.add.u64 [%0], %1;" ::"l"(p), "l"(v) : "memory");
}
// Programmatic dependent launch (kernels launched with the programmatic stream serialization
// attribute): launch_dependents lets the next such kernel in the stream start its CTAs while
// this grid still runs; wait returns once every grid this one depends on has completed and
// its writes are visible.  Both are no-ops for a plain launch.  Nothing written by an earlier
// launch (epoch, flags, status, data) may be read before the wait; descriptors are immutable.
__device__ __forceinline__ void pdl_launch_dependents() { asm volatile("griddepcontrol.launch_dependents;" ::: "memory"); }
__device__ __forceinline__ void pdl_wait() { asm volatile("griddepcontrol.wait;" ::: "memory"); }

__device__ __forceinline__ unsigned long long globaltimer_ns() {
  unsigned long long t;
  asm volatile("mov.u64 %0, %globaltimer;" : "=l"(t));
  return t;
}
__device__ __forceinline__ int ld_volatile_s32(const int* p) {
  int v;
  asm volatile("ld.volatile.global.s32 %0, [%1];" : "=r"(v) : "l"(p) : "memory");
  return v;
}
__device__ __forceinline__ uint4 ld16(const void* p) {
  uint4 v;
  asm volatile("ld.global.cg.v4.u32 {%0,%1,%2,%3}, [%4];" : "=r"(v.x), "=r"(v.y), "=r"(v.z), "=r"(v.w) : "l"(p));
  return v;
}
__device__ __forceinline__ void st16(void* p, const uint4& v) {
  asm volatile("st.global.cg.v4.u32 [%0], {%1,%2,%3,%4};" ::"l"(p), "r"(v.x), "r"(v.y), "r"(v.z), "r"(v.w) : "memory");
}

__device__ __forceinline__ char* resolve(const ExecParams& P, uint64_t packed) {
  return static_cast<char*>(P.base[packed >> 48]) + (packed & 0xFFFFFFFFFFFFull);
}
// The same for a schedule with two staging buffers: scratch addresses move by `scratch_shift`
// (0 or the distance to the second buffer, by launch parity); inputs and outputs stay.
__device__ __forceinline__ char* resolve(const ExecParams& P, uint64_t packed, unsigned long long scratch_shift) {
  const uint64_t slot = packed >> 48;
  return static_cast<char*>(P.base[slot]) + (packed & 0xFFFFFFFFFFFFull) +
         ((slot >= (uint64_t)kSlotScratch && slot < (uint64_t)kSlotAux) ? scratch_shift : 0ull);
}

// ---- element arithmetic ----------------------------------------------------------------
// A "unit" is the group of elements one 16-byte vector of the narrowest operand holds:
// 8 elements for bf16 schedules, 4 for fp32 / int32.
template <int DT>
struct Acc;

template <>
struct Acc<PL_BF16> {
  static constexpr int kElems = 8;
  float v[8];
  __device__ __forceinline__ void zero() {
#pragma unroll
    for (int i = 0; i < 8; ++i) v[i] = 0.f;
  }
  __device__ __forceinline__ void add_bf16(const uint4& q) {
    const uint32_t w[4] = {q.x, q.y, q.z, q.w};
#pragma unroll
    for (int i = 0; i < 4; ++i) {
      // fp32 += bf16 as one mixed-precision add per element (the bf16 operand is widened exactly,
      // the sum rounded to nearest once: bit for bit what shift / mask and an fp32 add give)
      uint16_t lo, hi;
      asm("mov.b32 {%0, %1}, %2;" : "=h"(lo), "=h"(hi) : "r"(w[i]));
      asm("add.rn.f32.bf16 %0, %1, %0;" : "+f"(v[2 * i]) : "h"(lo));
      asm("add.rn.f32.bf16 %0, %1, %0;" : "+f"(v[2 * i + 1]) : "h"(hi));
    }
  }
  __device__ __forceinline__ void add_f32(const uint4& lo, const uint4& hi) {
    v[0] += __uint_as_float(lo.x); v[1] += __uint_as_float(lo.y);
    v[2] += __uint_as_float(lo.z); v[3] += __uint_as_float(lo.w);
    v[4] += __uint_as_float(hi.x); v[5] += __uint_as_float(hi.y);
    v[6] += __uint_as_float(hi.z); v[7] += __uint_as_float(hi.w);
  }
  // final conversion; `scale` is the schedule's output scale (1 = plain sum, exact)
  __device__ __forceinline__ uint4 to_bf16(float scale = 1.0f) const {
    uint4 q;
    __nv_bfloat162 a = __floats2bfloat162_rn(v[0] * scale, v[1] * scale);
    __nv_bfloat162 b = __floats2bfloat162_rn(v[2] * scale, v[3] * scale);
    __nv_bfloat162 c = __floats2bfloat162_rn(v[4] * scale, v[5] * scale);
    __nv_bfloat162 d = __floats2bfloat162_rn(v[6] * scale, v[7] * scale);
    q.x = *reinterpret_cast<uint32_t*>(&a);
    q.y = *reinterpret_cast<uint32_t*>(&b);
    q.z = *reinterpret_cast<uint32_t*>(&c);
    q.w = *reinterpret_cast<uint32_t*>(&d);
    return q;
  }
};

// fp32 data: compensated (Kahan-Neumaier style two-sum) accumulation, still one
// accumulator per element and ascending source order; the correction is folded in once at
// the end.  Keeps the result inside the fp32 tolerance for any input mantissas.
template <>
struct Acc<PL_F32> {
  static constexpr int kElems = 4;
  float v[4], c[4];
  __device__ __forceinline__ void zero() {
#pragma unroll
    for (int i = 0; i < 4; ++i) v[i] = c[i] = 0.f;
  }
  __device__ __forceinline__ void add(const uint4& q) {
    const float x[4] = {__uint_as_float(q.x), __uint_as_float(q.y), __uint_as_float(q.z), __uint_as_float(q.w)};
#pragma unroll
    for (int i = 0; i < 4; ++i) {
      float s = __fadd_rn(v[i], x[i]);
      float bp = __fsub_rn(s, v[i]);
      float err = __fadd_rn(__fsub_rn(v[i], __fsub_rn(s, bp)), __fsub_rn(x[i], bp));
      c[i] = __fadd_rn(c[i], err);
      v[i] = s;
    }
  }
  // add a (sum, correction) pair: two-sum on the sums, corrections accumulate
  __device__ __forceinline__ void add_pair(const uint4& s, const uint4& corr) {
    add(s);
    c[0] = __fadd_rn(c[0], __uint_as_float(corr.x));
    c[1] = __fadd_rn(c[1], __uint_as_float(corr.y));
    c[2] = __fadd_rn(c[2], __uint_as_float(corr.z));
    c[3] = __fadd_rn(c[3], __uint_as_float(corr.w));
  }
  __device__ __forceinline__ uint4 sums() const {
    return make_uint4(__float_as_uint(v[0]), __float_as_uint(v[1]), __float_as_uint(v[2]), __float_as_uint(v[3]));
  }
  __device__ __forceinline__ uint4 corrections() const {
    return make_uint4(__float_as_uint(c[0]), __float_as_uint(c[1]), __float_as_uint(c[2]), __float_as_uint(c[3]));
  }
  __device__ __forceinline__ uint4 result(float scale = 1.0f) const {
    uint4 q;
    q.x = __float_as_uint(__fmul_rn(__fadd_rn(v[0], c[0]), scale));
    q.y = __float_as_uint(__fmul_rn(__fadd_rn(v[1], c[1]), scale));
    q.z = __float_as_uint(__fmul_rn(__fadd_rn(v[2], c[2]), scale));
    q.w = __float_as_uint(__fmul_rn(__fadd_rn(v[3], c[3]), scale));
    return q;
  }
};

template <>
struct Acc<PL_I32> {
  static constexpr int kElems = 4;
  uint32_t v[4];
  __device__ __forceinline__ void zero() { v[0] = v[1] = v[2] = v[3] = 0u; }
  __device__ __forceinline__ void add(const uint4& q) {
    v[0] += q.x; v[1] += q.y; v[2] += q.z; v[3] += q.w;
  }
  __device__ __forceinline__ uint4 result(float = 1.0f) const { return make_uint4(v[0], v[1], v[2], v[3]); }
};

// ---- processing phase of a final reduce op (Sec. 3.3: configurable while the sum is in registers)
// value = scale * sum [+ residual], then one conversion to the element type, or none (fp32 out).
// `dst` points at this unit in the destination (16 bytes per unit; 32 for fp32 output of a bf16
// schedule), `res` at the same unit of the second operand (element-typed) or is unused.
// `q` is the unit of the second operand, already loaded (ignored without PL_HOOK_RESIDUAL).
// final_value computes the unit's result: 16 bytes in `lo`, or 32 bytes in `lo`, `hi` for the
// fp32 output of a bf16 schedule (returns true then).
template <int DT>
__device__ __forceinline__ bool final_value(const Acc<DT>& acc, float scale, uint32_t hook, const uint4& q, uint4& lo, uint4& hi) {
  if constexpr (DT == PL_BF16) {
    float v[8];
#pragma unroll
    for (int i = 0; i < 8; ++i) v[i] = __fmul_rn(acc.v[i], scale);
    if (hook & PL_HOOK_RESIDUAL) {
      const uint32_t w[4] = {q.x, q.y, q.z, q.w};
#pragma unroll
      for (int i = 0; i < 4; ++i) {
        v[2 * i] = __fadd_rn(v[2 * i], __uint_as_float(w[i] << 16));
        v[2 * i + 1] = __fadd_rn(v[2 * i + 1], __uint_as_float(w[i] & 0xFFFF0000u));
      }
    }
    if (hook & PL_HOOK_F32_OUT) {
      lo = make_uint4(__float_as_uint(v[0]), __float_as_uint(v[1]), __float_as_uint(v[2]), __float_as_uint(v[3]));
      hi = make_uint4(__float_as_uint(v[4]), __float_as_uint(v[5]), __float_as_uint(v[6]), __float_as_uint(v[7]));
      return true;
    }
    __nv_bfloat162 a = __floats2bfloat162_rn(v[0], v[1]), b = __floats2bfloat162_rn(v[2], v[3]);
    __nv_bfloat162 c = __floats2bfloat162_rn(v[4], v[5]), d = __floats2bfloat162_rn(v[6], v[7]);
    lo.x = *reinterpret_cast<uint32_t*>(&a);
    lo.y = *reinterpret_cast<uint32_t*>(&b);
    lo.z = *reinterpret_cast<uint32_t*>(&c);
    lo.w = *reinterpret_cast<uint32_t*>(&d);
    return false;
  } else if constexpr (DT == PL_F32) {
    float v[4];
#pragma unroll
    for (int i = 0; i < 4; ++i) v[i] = __fmul_rn(__fadd_rn(acc.v[i], acc.c[i]), scale);
    if (hook & PL_HOOK_RESIDUAL) {
      v[0] = __fadd_rn(v[0], __uint_as_float(q.x));
      v[1] = __fadd_rn(v[1], __uint_as_float(q.y));
      v[2] = __fadd_rn(v[2], __uint_as_float(q.z));
      v[3] = __fadd_rn(v[3], __uint_as_float(q.w));
    }
    lo = make_uint4(__float_as_uint(v[0]), __float_as_uint(v[1]), __float_as_uint(v[2]), __float_as_uint(v[3]));
    return false;
  } else {
    return false;
  }
}

template <int DT>
__device__ __forceinline__ void store_final_q(const Acc<DT>& acc, float scale, uint32_t hook, char* dst, const uint4& q) {
  uint4 lo, hi;
  const bool wide = final_value<DT>(acc, scale, hook, q, lo, hi);
  st16(dst, lo);
  if (wide) st16(dst + 16, hi);
}

template <int DT>
__device__ __forceinline__ void store_final(const Acc<DT>& acc, float scale, uint32_t hook, char* dst, const char* res) {
  uint4 q = make_uint4(0, 0, 0, 0);
  if (hook & PL_HOOK_RESIDUAL) q = ld16(res);
  store_final_q<DT>(acc, scale, hook, dst, q);
}

// A final op of a hooked schedule stores unit `unit` of its result to one destination or to all
// ranks' outputs.  dst_packed = (slot << 48) | byte offset of the op's destination; the second
// operand of rank k sits in slot kSlotAux + k, laid out like the (element-typed) output.
template <int DT>
__device__ __forceinline__ void store_final_unit(const ExecParams& P, const Acc<DT>& acc, uint64_t dst_slot, uint64_t dst_off,
                                                 bool bcast, uint64_t unit) {
  const uint32_t hook = P.hook;
  const bool f32 = (DT == PL_BF16) && (hook & PL_HOOK_F32_OUT);
  const uint64_t d_off = dst_off + unit * (f32 ? 32ull : 16ull);       // bytes into the output
  const uint64_t r_off = (f32 ? dst_off >> 1 : dst_off) + unit * 16ull;  // bytes into the second operand
  if (!bcast) {
    const char* res = (hook & PL_HOOK_RESIDUAL) ? static_cast<const char*>(P.base[kSlotAux + (dst_slot - kSlotOut)]) + r_off : nullptr;
    store_final<DT>(acc, P.out_scale, hook, static_cast<char*>(P.base[dst_slot]) + d_off, res);
  } else {
    for (int k = 0; k < P.n_ranks; ++k) {
      const char* res = (hook & PL_HOOK_RESIDUAL) ? static_cast<const char*>(P.base[kSlotAux + k]) + r_off : nullptr;
      store_final<DT>(acc, P.out_scale, hook, static_cast<char*>(P.base[kSlotOut + k]) + d_off, res);
    }
  }
}

// ---- SM-window launches -------------------------------------------------------------------
// One CTA is launched per SM; a CTA whose SM lies in the idle window (bit clear in `mask`, one bit
// per SM id, 160 bits) sits the launch out, every other CTA claims the next of n_slots work slots
// (op queues of a schedule, strides of a stream).  How fast a 1 read : R writes stream runs depends
// on WHICH SMs take part (see pl_comm_tune), and a plain launch of fewer CTAs than SMs leaves that
// choice to the hardware.
// State (three 64-bit words, zero between launches): [0] arrivals << 32 | slots claimed by CTAs on
// active SMs, [1] slots claimed afterwards, [2] CTAs that have left.  Every CTA adds itself to [0]
// with ONE atomic (no compare-and-swap loop: 148 CTAs contending for one word would take tens of
// microseconds).  A CTA on an active SM takes the slot it drew.  A CTA on an idle SM waits until
// all CTAs have arrived, normally a microsecond, and leaves; should the CTAs not have landed one
// per SM (other work on the GPU), slots are left over then and the waiting CTAs draw them from
// [1], so every slot is taken exactly once.  The last CTA to leave zeroes the state.
// Returns the slot, or -1 (nothing to do).  *timed_out: arrivals still incomplete after limit_ns.
__device__ __forceinline__ int window_claim(unsigned long long* state, const uint32_t* mask, uint32_t n_slots,
                                            unsigned long long limit_ns, bool* timed_out) {
  uint32_t sm;
  asm volatile("mov.u32 %0, %%smid;" : "=r"(sm));
  const bool active = sm >= 160u || ((mask[sm >> 5] >> (sm & 31u)) & 1u);
  const uint32_t total = gridDim.x;
  const unsigned long long mine = (1ull << 32) | (active ? 1ull : 0ull);
  const unsigned long long old = atomicAdd(state, mine);
  if (active) {
    const uint32_t taken = (uint32_t)old;
    return taken < n_slots ? (int)taken : -1;  // a surplus CTA on an active SM has nothing to do
  }
  unsigned long long now = old + mine;
  const unsigned long long t0 = globaltimer_ns();
  for (uint32_t spins = 1; (uint32_t)(now >> 32) < total; ++spins) {
    now = *reinterpret_cast<volatile unsigned long long*>(state);
    if ((spins & 63u) == 0 && globaltimer_ns() - t0 > limit_ns) break;
  }
  if ((uint32_t)(now >> 32) < total) {
    *timed_out = true;
    return -1;
  }
  const uint32_t by_active = (uint32_t)now;
  if (by_active >= n_slots) return -1;
  const uint32_t extra = atomicAdd(reinterpret_cast<unsigned int*>(state + 1), 1u);
  return by_active + extra < n_slots ? (int)(by_active + extra) : -1;
}
// A CTA of an SM-window launch leaves: the last one puts the state back to zero.
__device__ __forceinline__ void window_leave(unsigned long long* state) {
  __threadfence();
  const unsigned int left = atomicAdd(reinterpret_cast<unsigned int*>(state + 2), 1u);
  if (left == gridDim.x - 1u) {
    state[0] = 0ull;
    state[1] = 0ull;
    state[2] = 0ull;
    __threadfence();
  }
}

// Record a timeout (first writer wins) and raise the abort word.
static __device__ __noinline__ void record_timeout_at(int* status, int queue, uint32_t topo, uint32_t flag,
                                                      unsigned long long expected, unsigned long long observed) {
  if (atomicCAS(status, 0, (int)PL_ERR_TIMEOUT) == 0) {
    status[1] = queue;
    status[2] = (int)topo;
    status[3] = (int)flag;
    *reinterpret_cast<unsigned long long*>(status + 4) = expected;
    *reinterpret_cast<unsigned long long*>(status + 6) = observed;
  }
  __threadfence();
  atomicExch(status + 8, 1);
}
static __device__ __forceinline__ void record_timeout(const ExecParams& P, int queue, uint32_t topo, uint32_t flag,
                                                      unsigned long long expected, unsigned long long observed) {
  record_timeout_at(P.status, queue, topo, flag, expected, observed);
}

}  // namespace dev
}  // namespace pl
