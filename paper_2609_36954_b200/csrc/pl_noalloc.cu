// pl_reduce_scatter_ring_static: a ring reduce-scatter that allocates nothing.
//
// Written for callers that are not allowed to allocate device memory at the point where they
// need a collective: code running inside a memory-pool or arena discipline where every byte is
// planned up front, a latency-critical serving loop where cudaMalloc's implicit device
// synchronisation is unacceptable, or a plugin that is handed input and output buffers and
// nothing else.  The ring algorithm needs room for the partial sums that travel between ranks;
// here that room is a fixed array compiled into the library image, so the entry point only
// launches one kernel.
//
// The price: the array has a fixed size (kScratchBytes per GPU, resident from the moment the
// library is loaded on that GPU until the process exits), so messages beyond what fits are
// refused; and all calls on a GPU share it, so two calls that overlap in time on the same GPU
// (different streams) would overwrite each other's partial sums.  Nothing in it has to start
// at zero: partial sums are fully rewritten by every call, and the readiness words carry a
// call number that only grows, so left-overs of earlier calls are never mistaken for "ready".
// The call number lives on the device (every CTA reads it at entry, the last CTA to leave
// advances it), so it follows the order in which the launches actually run: host threads that
// enqueue in another order than they entered, or a captured launch that is replayed, cannot
// desynchronise it.
#include <cuda_runtime.h>

#include <atomic>
#include <mutex>

#include "pl_api_internal.h"
#include "pl_device.cuh"
#include "pl_internal.h"

using namespace pl;
using namespace pl::dev;

namespace {

constexpr size_t kScratchBytes = 32u << 20;  // partial sums of all ranks and steps
constexpr int kMaxSlices = 16;               // CTAs per rank
constexpr int kMaxDevices = 64;
constexpr int kThreads = 512;

// Device-resident state.  In host code these names are only handles for the runtime: the
// device addresses are looked up once per device with cudaGetSymbolAddress (see setup()).
static __device__ __align__(256) unsigned char g_scratch[kScratchBytes];
static __device__ __align__(256) unsigned long long g_ready[PL_MAX_RANKS * PL_MAX_RANKS * kMaxSlices];
static __device__ __align__(256) unsigned long long g_calls[2];  // [0] calls completed, [1] CTAs of the running call that left

struct RingParams {
  const void* in[PL_MAX_RANKS];
  void* out[PL_MAX_RANKS];
  unsigned char* scratch;       // device address of g_scratch
  unsigned long long* ready;    // device address of g_ready: [rank][step][slice]
  int* status;                  // caller-owned device word (may be null): 0 or PL_ERR_TIMEOUT
  unsigned long long* calls;    // device address of g_calls
  unsigned long long wait_bias; // 0; the test hook raises what every wait expects so that it can never be met
  unsigned long long units;     // 16-byte units of the element type per partition
  unsigned long long timeout_ns;
  int R;
};

// dst = a + b over `n` units starting at unit `first`; a and dst may hold partials.
template <int DT>
__device__ __forceinline__ void add_slice(char* dst, bool dpart, const char* a, bool apart, const char* b,
                                          unsigned long long first, unsigned long long n, int tid) {
  for (unsigned long long i = first + tid; i < first + n; i += kThreads) {
    Acc<DT> acc;
    acc.zero();
    if constexpr (DT == PL_BF16) {
      if (apart) acc.add_f32(ld16(a + (i << 5)), ld16(a + (i << 5) + 16));
      else acc.add_bf16(ld16(a + (i << 4)));
      acc.add_bf16(ld16(b + (i << 4)));
      if (dpart) {
        st16(dst + (i << 5), make_uint4(__float_as_uint(acc.v[0]), __float_as_uint(acc.v[1]), __float_as_uint(acc.v[2]), __float_as_uint(acc.v[3])));
        st16(dst + (i << 5) + 16, make_uint4(__float_as_uint(acc.v[4]), __float_as_uint(acc.v[5]), __float_as_uint(acc.v[6]), __float_as_uint(acc.v[7])));
      } else {
        st16(dst + (i << 4), acc.to_bf16());
      }
    } else if constexpr (DT == PL_F32) {
      if (apart) acc.add_pair(ld16(a + (i << 5)), ld16(a + (i << 5) + 16));
      else acc.add(ld16(a + (i << 4)));
      acc.add(ld16(b + (i << 4)));
      if (dpart) {
        st16(dst + (i << 5), acc.sums());
        st16(dst + (i << 5) + 16, acc.corrections());
      } else {
        st16(dst + (i << 4), acc.result());
      }
    } else {
      acc.add(ld16(a + (i << 4)));
      acc.add(ld16(b + (i << 4)));
      st16(dst + (i << 4), acc.result());
    }
  }
}

// grid (slices, R): CTA (g, r) runs slice g of every step of rank r.  Step s of rank r adds
// rank r's input partition k = (r - s - 2) mod R to what rank r-1 produced in step s-1 (rank
// r-1's own input in step 0); the last step writes rank r's output.
template <int DT>
__global__ void __launch_bounds__(kThreads) pl_ring_rs_static_kernel(const __grid_constant__ RingParams p) {
  __shared__ int s_abort;
  const int g = blockIdx.x, G = gridDim.x, r = blockIdx.y, R = p.R, tid = threadIdx.x;
  constexpr int es = (DT == PL_BF16) ? 2 : 4;
  constexpr int ps = (DT == PL_BF16) ? 4 : (DT == PL_F32 ? 8 : 4);  // bytes per element of a partial
  constexpr int kE = Acc<DT>::kElems;
  const unsigned long long U = p.units, first = U * g / G, n = U * (g + 1) / G - first;
  const unsigned long long part_e = U * kE;  // elements per partition
  const int q = (r + R - 1) % R;
  if (tid == 0) s_abort = 0;
  // number of this call: all CTAs read the counter before any of them reports that it has left,
  // and it only moves once all of them have, so they agree
  const unsigned long long call = *reinterpret_cast<volatile unsigned long long*>(p.calls) + 1ull;
  const unsigned long long expect = call + p.wait_bias;
  __syncthreads();
  bool aborted = false;
  for (int s = 0; s <= R - 2; ++s) {
    const int k = ((r - s - 2) % R + R) % R;
    const bool last = s == R - 2;
    if (s > 0 && tid == 0) {
      const unsigned long long* f = p.ready + ((size_t)q * PL_MAX_RANKS + (s - 1)) * kMaxSlices + g;
      if (ld_acquire_u64(f) < expect) {
        const unsigned long long t0 = globaltimer_ns();
        unsigned spins = 0;
        while (ld_acquire_u64(f) < expect) {
          if ((++spins & 63u) == 0 && globaltimer_ns() - t0 > p.timeout_ns) {
            if (p.status) atomicExch(p.status, (int)PL_ERR_TIMEOUT);
            s_abort = 1;
            break;
          }
        }
      }
    }
    __syncthreads();
    if (s_abort) { aborted = true; break; }
    const char* a = (s == 0) ? static_cast<const char*>(p.in[q]) + (size_t)k * part_e * es
                             : reinterpret_cast<const char*>(p.scratch) + ((size_t)q * (R - 2) + (s - 1)) * part_e * ps;
    const char* b = static_cast<const char*>(p.in[r]) + (size_t)k * part_e * es;
    char* d = last ? static_cast<char*>(p.out[r])
                   : reinterpret_cast<char*>(p.scratch) + ((size_t)r * (R - 2) + s) * part_e * ps;
    add_slice<DT>(d, !last, a, s > 0, b, first, n, tid);
    if (!last) {
      __syncthreads();
      if (tid == 0) {
        __threadfence();
        asm volatile("st.release.gpu.global.u64 [%0], %1;" ::"l"(p.ready + ((size_t)r * PL_MAX_RANKS + s) * kMaxSlices + g), "l"(call) : "memory");
      }
    }
  }
  (void)aborted;
  // The last CTA to leave advances the call number, after a timeout too: the next call then
  // expects a larger number than anything this one may have left in the readiness words.
  __syncthreads();
  if (tid == 0) {
    const unsigned long long left = atomicAdd(p.calls + 1, 1ull);
    if (left == (unsigned long long)gridDim.x * gridDim.y - 1ull) {
      p.calls[1] = 0ull;
      __threadfence();
      *reinterpret_cast<volatile unsigned long long*>(p.calls) = call;
    }
  }
}

struct DeviceState {
  bool ready = false;
  unsigned char* scratch = nullptr;
  unsigned long long* flags = nullptr;
  unsigned long long* calls = nullptr;
  int sm_count = 0;
};
DeviceState g_dev[kMaxDevices];
std::mutex g_mu;

// Once per device, with that device current: turn the symbols into device addresses.
pl_status_t setup(int device, DeviceState** out) {
  if (device < 0 || device >= kMaxDevices) return PL_ERR_INVALID_ARG;
  DeviceState& d = g_dev[device];
  if (!d.ready) {
    if (cudaGetSymbolAddress(reinterpret_cast<void**>(&d.scratch), g_scratch) != cudaSuccess ||
        cudaGetSymbolAddress(reinterpret_cast<void**>(&d.flags), g_ready) != cudaSuccess ||
        cudaGetSymbolAddress(reinterpret_cast<void**>(&d.calls), g_calls) != cudaSuccess ||
        cudaDeviceGetAttribute(&d.sm_count, cudaDevAttrMultiProcessorCount, device) != cudaSuccess) {
      cudaGetLastError();
      return PL_ERR_CUDA;
    }
    d.ready = true;
  }
  *out = &d;
  return PL_OK;
}

}  // namespace

static pl_status_t ring_static(int R, pl_dtype_t dtype, size_t count_per_rank, const void* const* in, void* const* out,
                               int32_t* status, void* stream, unsigned long long wait_bias, unsigned long long timeout_ns) {
  if (R < 2 || R > PL_MAX_RANKS || !in || !out) return PL_ERR_INVALID_ARG;
  if (dtype != PL_BF16 && dtype != PL_F32 && dtype != PL_I32) return PL_ERR_UNSUPPORTED;
  const size_t es = elem_size(dtype), ps = elem_size(partial_dtype(dtype));
  if (count_per_rank == 0 || (count_per_rank * es) % (16u * R)) return PL_ERR_INVALID_ARG;
  const size_t part = count_per_rank / R;  // elements per partition
  if (R > 2 && (size_t)R * (R - 2) * part * ps > kScratchBytes) return PL_ERR_OVERFLOW;
  for (int r = 0; r < R; ++r) {
    if (!in[r] || !out[r]) return PL_ERR_INVALID_ARG;
    if (((uintptr_t)in[r] & 15) || ((uintptr_t)out[r] & 15)) return PL_ERR_ALIGNMENT;
  }
  int device = -1;
  if (cudaGetDevice(&device) != cudaSuccess) { cudaGetLastError(); return PL_ERR_CUDA; }
  RingParams p;
  DeviceState* d = nullptr;
  // one caller at a time from set-up to launch: calls reach the stream in the order they got here
  std::lock_guard<std::mutex> lock(g_mu);
  pl_status_t st = setup(device, &d);
  if (st != PL_OK) return st;
  for (int r = 0; r < PL_MAX_RANKS; ++r) {
    p.in[r] = r < R ? in[r] : nullptr;
    p.out[r] = r < R ? out[r] : nullptr;
  }
  p.scratch = d->scratch;
  p.ready = d->flags;
  p.calls = d->calls;
  p.wait_bias = wait_bias;
  p.status = status;
  p.units = part * es / 16;
  p.timeout_ns = timeout_ns;
  p.R = R;
  // all CTAs wait on one another, so the grid must be co-resident: at most one CTA per SM
  int slices = d->sm_count / R;
  if (slices > kMaxSlices) slices = kMaxSlices;
  if ((unsigned long long)slices > p.units) slices = (int)p.units;
  if (slices < 1) return PL_ERR_OVERSUBSCRIBED;
  dim3 grid(slices, R);
  cudaStream_t cs = static_cast<cudaStream_t>(stream);
  if (status && cudaMemsetAsync(status, 0, sizeof(int32_t), cs) != cudaSuccess) { cudaGetLastError(); return PL_ERR_CUDA; }
  switch (dtype) {
    case PL_BF16: pl_ring_rs_static_kernel<PL_BF16><<<grid, kThreads, 0, cs>>>(p); break;
    case PL_F32: pl_ring_rs_static_kernel<PL_F32><<<grid, kThreads, 0, cs>>>(p); break;
    default: pl_ring_rs_static_kernel<PL_I32><<<grid, kThreads, 0, cs>>>(p); break;
  }
  if (cudaGetLastError() != cudaSuccess) return PL_ERR_CUDA;
  g_launches.fetch_add(1);
  return PL_OK;
}

extern "C" pl_status_t pl_reduce_scatter_ring_static(int R, pl_dtype_t dtype, size_t count_per_rank,
                                                     const void* const* in, void* const* out,
                                                     int32_t* status, void* stream) {
  return ring_static(R, dtype, count_per_rank, in, out, status, stream, 0ull, 2000000000ull);
}

// TEST HOOK: the same call, but every wait inside the kernel expects a call number that is never
// published and gives up after timeout_ns, so that the time-out path (status word set, kernel
// returns, later calls work) can be exercised without hanging a GPU.
extern "C" pl_status_t pl_reduce_scatter_ring_static_debug_timeout(int R, pl_dtype_t dtype, size_t count_per_rank,
                                                                   const void* const* in, void* const* out,
                                                                   int32_t* status, void* stream, uint64_t timeout_ns) {
  if (timeout_ns == 0 || timeout_ns > 1000000000ull) return PL_ERR_INVALID_ARG;
  return ring_static(R, dtype, count_per_rank, in, out, status, stream, 1ull << 40, timeout_ns);
}
