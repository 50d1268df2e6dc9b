// Packet datapath: the latency specialisation of the paper (Sec. 3.2, "Specializing for
// latency").  L back-to-back one-shot all-reduces of a small message run in one launch.
//
// A packet is 16 bytes: 8 bytes of payload and an 8-byte tag that travel in one store and one
// load, so data and "data is ready" arrive together and no separate flag word, fence or acquire
// sits on the path.  A thread owns 16 bytes of the message, i.e. two neighbouring packets (one
// 32-byte sector), and moves both with one 256-bit access; each packet carries its own tag and
// both tags are checked.  The tag is the global layer number (executes
// completed * L + layer + 1): it only grows, nothing is ever reset, and a consumer accepts a
// packet only when the tag is exactly the one it expects.
//
// Rank r is a thread-block cluster of G CTAs.  Per layer l every CTA
//   1. polls, for its slice of the message, the packets of all R ranks (ascending rank order,
//      fp32 accumulation, one conversion: Eq. "rank-order") and stores its slice of out[r];
//   2. joins the other CTAs of its rank with a cluster barrier: rank r's layer-l output is
//      complete (the rule that a rank may not publish layer l+1 before that);
//   3. publishes its slice of rank r's layer-(l+1) input as packets (the payload was fetched
//      into registers beforehand: inputs are constant, only the publication is ordered).
// Ranks share one memory here, so a producer writes ONE copy of its packets and all consumers
// read it (across GPUs the paper pushes a copy into every consumer's buffer).  Packets of
// even and odd global layers live in two buffers: a rank publishes layer l+2 only after it has
// consumed layer l+1 of every rank, which they published after consuming layer l, so nobody
// still reads the buffer that is being overwritten (the paper's epoch-parity double
// buffering, Sec. 4.2).
//
// Every poll is bounded: on expiry the thread records the time-out, raises the abort word and
// keeps walking through the remaining barriers without polling, so the cluster never hangs.
#include <cuda_bf16.h>
#include <cuda_runtime.h>

#include <atomic>

#include "pl_device.cuh"
#include "pl_internal.h"
#include "pl_kernels.h"

namespace pl {
namespace {

using namespace dev;

constexpr int kMaxUnitsPerThread = 4;  // 16-byte output vectors one thread owns per layer
constexpr int kBatch = 8;              // sources polled at once (two packets each)
constexpr int kMaxThreads = 256;       // 64 registers of packets in flight per thread

struct Packet {
  unsigned long long payload, tag;
};

__device__ __forceinline__ Packet ld_packet(const void* p) {
  Packet k;
  asm volatile("ld.relaxed.gpu.global.v2.u64 {%0,%1}, [%2];" : "=l"(k.payload), "=l"(k.tag) : "l"(p) : "memory");
  return k;
}
// Two neighbouring packets (one 32-byte sector) with one 256-bit access.
struct Packet2 {
  Packet lo, hi;
};
__device__ __forceinline__ Packet2 ld_packet2(const void* p) {
  Packet2 k;
  asm volatile("ld.relaxed.gpu.global.v4.u64 {%0,%1,%2,%3}, [%4];"
               : "=l"(k.lo.payload), "=l"(k.lo.tag), "=l"(k.hi.payload), "=l"(k.hi.tag)
               : "l"(p)
               : "memory");
  return k;
}
__device__ __forceinline__ void st_packet2(void* p, unsigned long long pay0, unsigned long long pay1, unsigned long long tag) {
  asm volatile("st.relaxed.gpu.global.v4.u64 [%0], {%1,%2,%3,%4};" ::"l"(p), "l"(pay0), "l"(tag), "l"(pay1), "l"(tag) : "memory");
}
__device__ __forceinline__ void cluster_arrive() { asm volatile("barrier.cluster.arrive.release.aligned;" ::: "memory"); }
__device__ __forceinline__ void cluster_wait() { asm volatile("barrier.cluster.wait.acquire.aligned;" ::: "memory"); }

template <int DT>
__global__ void __launch_bounds__(kMaxThreads) pl_exec_packet_kernel(const __grid_constant__ PacketParams P) {
  __shared__ int s_abort;
  const int tid = threadIdx.x, nthr = blockDim.x;
  const int G = P.ctas_per_rank, r = blockIdx.x / G, j = blockIdx.x % G;
  const int R = P.n_ranks, L = P.n_layers;
  const uint64_t UC = P.units_per_rank / (uint64_t)G;  // 16-byte vectors of the message this CTA owns
  const uint64_t u0 = (uint64_t)j * UC;
  const uint64_t msg = P.units_per_rank * 16ull;       // bytes of one layer's message
  const uint64_t half = P.units_per_rank * 32ull;      // bytes of one packet buffer (one parity)
  pdl_launch_dependents();
  if (tid == 0) s_abort = 0;
  pdl_wait();
  const unsigned long long epoch = *reinterpret_cast<volatile unsigned long long*>(P.epoch);
  const unsigned long long gl0 = epoch * (unsigned long long)L;
  __syncthreads();

  // this thread's vectors: u0 + tid + k * nthr, k < kMaxUnitsPerThread (build guarantees the bound)
  uint4 pub[kMaxUnitsPerThread];
  auto fetch_pub = [&](int layer) {
#pragma unroll
    for (int k = 0; k < kMaxUnitsPerThread; ++k) {
      const uint64_t u = (uint64_t)tid + (uint64_t)k * nthr;
      if (u < UC) pub[k] = ld16(static_cast<const char*>(P.in[r]) + (uint64_t)layer * msg + (u0 + u) * 16ull);
    }
  };
  auto publish = [&](unsigned long long gl) {
    char* base = static_cast<char*>(P.pkt[r]) + (gl & 1ull) * half;
#pragma unroll
    for (int k = 0; k < kMaxUnitsPerThread; ++k) {
      const uint64_t u = (uint64_t)tid + (uint64_t)k * nthr;
      if (u < UC) {
        char* at = base + (u0 + u) * 32ull;
        st_packet2(at, ((unsigned long long)pub[k].y << 32) | pub[k].x, ((unsigned long long)pub[k].w << 32) | pub[k].z, gl + 1ull);
      }
    }
  };

  fetch_pub(0);
  publish(gl0);
  bool aborted = false;
  for (int l = 0; l < L; ++l) {
    const unsigned long long gl = gl0 + (unsigned long long)l;
    // test hook: the op named by break_op expects a tag nobody publishes
    const unsigned long long want = gl + 1ull + (((long long)l * R + r) * G + j == P.break_op ? (1ull << 40) : 0ull);
    if (l + 1 < L) fetch_pub(l + 1);
    if (!aborted) {
      const int lane = tid & 31;
#pragma unroll 1
      for (int k = 0; k < kMaxUnitsPerThread; ++k) {
        // control flow is uniform per warp from here to the end of the iteration
        const uint64_t warp_first = (uint64_t)(tid & ~31) + (uint64_t)k * nthr;  // this warp's first vector
        if (warp_first >= UC) break;
        const uint64_t u = (uint64_t)tid + (uint64_t)k * nthr;
        const bool mine = u < UC;
        // ---- watch one packet per source first.  Polling every packet of every thread re-reads
        // the whole message per round: that is bound by the SM's L2 bandwidth, not by latency,
        // and the flood of loads delays the very stores it waits for.  The warp that publishes
        // this warp's vectors for rank p is the same warp of the same CTA index in rank p, and
        // the last packet it stores is the second packet of its last lane: lane p polls that one
        // packet of rank p.  When all R are there, the full read below almost always finds
        // everything in place (and polls on for whatever is not).
        {
          const uint64_t warp_last = min(UC - 1, warp_first + 31);
          const bool poller = lane < R;
          const char* sentinel = static_cast<const char*>(P.pkt[poller ? lane : 0]) + (gl & 1ull) * half + (u0 + warp_last) * 32ull + 16;
          bool here = !poller || ld_packet(sentinel).tag == want;
          if (!__all_sync(0xFFFFFFFFu, here)) {
            const unsigned long long t0 = globaltimer_ns();
            uint32_t spins = 0;
            for (;;) {
              if (!here) here = ld_packet(sentinel).tag == want;
              if (__all_sync(0xFFFFFFFFu, here)) break;
              if ((++spins & 63u) == 0) {
                bool give_up = ld_volatile_s32(P.status + 8) != 0;
                if (!give_up && !here && globaltimer_ns() - t0 > P.timeout_ns) {
                  record_timeout_at(P.status, blockIdx.x, (uint32_t)((l * R + r) * G + j), (uint32_t)lane, want,
                                    ld_packet(sentinel).tag);
                  give_up = true;
                }
                if (__any_sync(0xFFFFFFFFu, give_up)) { aborted = true; break; }
              }
            }
          }
        }
        if (aborted) break;  // warp-uniform
        if (P.trace && tid == 0 && k == 0) P.trace[2 * (((uint64_t)l * R + r) * G + j)] = globaltimer_ns();  // sentinels of every rank seen
        Acc<DT> acc;
        acc.zero();
        const uint64_t at = (gl & 1ull) * half + (u0 + u) * 32ull;
        bool failed = false;
#pragma unroll 1
        for (int p0 = 0; p0 < R && mine && !failed; p0 += kBatch) {
          Packet lo[kBatch], hi[kBatch];
          uint32_t pending = 0;
#pragma unroll
          for (int b = 0; b < kBatch; ++b)
            if (p0 + b < R) {
              const Packet2 two = ld_packet2(static_cast<const char*>(P.pkt[p0 + b]) + at);
              lo[b] = two.lo;
              hi[b] = two.hi;
            }
#pragma unroll
          for (int b = 0; b < kBatch; ++b)
            if (p0 + b < R && (lo[b].tag != want || hi[b].tag != want)) pending |= 1u << b;
          if (pending) {
            const unsigned long long t0 = globaltimer_ns();
            uint32_t spins = 0;
            while (pending) {
              // all missing packets are asked for again before any answer is looked at: one
              // round trip per round, not one per source
#pragma unroll
              for (int b = 0; b < kBatch; ++b)
                if ((pending >> b) & 1u) {
                  const Packet2 two = ld_packet2(static_cast<const char*>(P.pkt[p0 + b]) + at);
                  lo[b] = two.lo;
                  hi[b] = two.hi;
                }
#pragma unroll
              for (int b = 0; b < kBatch; ++b)
                if (((pending >> b) & 1u) && lo[b].tag == want && hi[b].tag == want) pending &= ~(1u << b);
              if (pending && (++spins & 63u) == 0) {
                if (ld_volatile_s32(P.status + 8)) { failed = true; break; }
                if (globaltimer_ns() - t0 > P.timeout_ns) {
                  const int first = __ffs(pending) - 1;  // the lowest rank whose packets are missing
                  unsigned long long seen = 0;
#pragma unroll
                  for (int b = 0; b < kBatch; ++b)
                    if (b == first) seen = lo[b].tag != want ? lo[b].tag : hi[b].tag;
                  record_timeout_at(P.status, blockIdx.x, (uint32_t)((l * R + r) * G + j), (uint32_t)(p0 + first), want, seen);
                  failed = true;
                  break;
                }
              }
            }
          }
          if (!failed) {
#pragma unroll
            for (int b = 0; b < kBatch; ++b)
              if (p0 + b < R) {
                const uint4 q = make_uint4((uint32_t)lo[b].payload, (uint32_t)(lo[b].payload >> 32),
                                           (uint32_t)hi[b].payload, (uint32_t)(hi[b].payload >> 32));
                if constexpr (DT == PL_BF16) acc.add_bf16(q);
                else acc.add(q);
              }
          }
        }
        if (mine && !failed) {
          uint4 res;
          if constexpr (DT == PL_BF16) res = acc.to_bf16(P.out_scale);
          else res = acc.result(P.out_scale);
          st16(static_cast<char*>(P.out[r]) + (uint64_t)l * msg + (u0 + u) * 16ull, res);
        }
        if (__any_sync(0xFFFFFFFFu, failed)) { aborted = true; break; }
      }
      if (aborted) s_abort = 1;
    }
    if (P.trace) {
      __syncthreads();
      if (tid == 0) {
        // about to join: every thread has read its packets and stored its part of the slice
        P.trace[2 * (((uint64_t)l * R + r) * G + j) + 1] = globaltimer_ns();
      }
    }
    // ---- join: rank r's layer-l output is complete when every CTA of the rank is here
    if (G > 1) {
      cluster_arrive();
      cluster_wait();
    } else {
      __syncthreads();
    }
    if (*reinterpret_cast<volatile int*>(&s_abort)) aborted = true;
    if (l + 1 < L && !aborted) publish(gl + 1ull);
  }

  __syncthreads();
  if (tid == 0 && !*reinterpret_cast<volatile int*>(&s_abort)) {
    const unsigned long long prev = atomicAdd(P.epoch + 1, 1ull);
    if (prev == (unsigned long long)gridDim.x - 1ull) {
      P.epoch[1] = 0ull;
      __threadfence();
      *reinterpret_cast<volatile unsigned long long*>(P.epoch) = epoch + 1ull;
    }
  }
}

template <int DT>
cudaError_t launch_t(const PacketParams& P, int threads, bool overlap, cudaStream_t stream) {
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = dim3((unsigned)(P.n_ranks * P.ctas_per_rank));
  cfg.blockDim = dim3((unsigned)threads);
  cfg.stream = stream;
  cudaLaunchAttribute attr[2];
  int na = 0;
  if (P.ctas_per_rank > 1) {
    attr[na].id = cudaLaunchAttributeClusterDimension;
    attr[na].val.clusterDim.x = (unsigned)P.ctas_per_rank;
    attr[na].val.clusterDim.y = 1;
    attr[na].val.clusterDim.z = 1;
    ++na;
  }
  if (overlap) {
    attr[na].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[na].val.programmaticStreamSerializationAllowed = 1;
    ++na;
  }
  cfg.attrs = attr;
  cfg.numAttrs = na;
  return cudaLaunchKernelEx(&cfg, pl_exec_packet_kernel<DT>, P);
}

template <int DT>
int clusters_t(int ctas_per_rank, int threads) {
  if (ctas_per_rank <= 1) {
    int n = 0, sms = 0, dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess || cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess ||
        cudaOccupancyMaxActiveBlocksPerMultiprocessor(&n, pl_exec_packet_kernel<DT>, threads, 0) != cudaSuccess) {
      cudaGetLastError();
      return 0;
    }
    return n * sms;
  }
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = dim3((unsigned)ctas_per_rank);
  cfg.blockDim = dim3((unsigned)threads);
  cudaLaunchAttribute attr[1];
  attr[0].id = cudaLaunchAttributeClusterDimension;
  attr[0].val.clusterDim.x = (unsigned)ctas_per_rank;
  attr[0].val.clusterDim.y = 1;
  attr[0].val.clusterDim.z = 1;
  cfg.attrs = attr;
  cfg.numAttrs = 1;
  int n = 0;
  if (cudaOccupancyMaxActiveClusters(&n, pl_exec_packet_kernel<DT>, &cfg) != cudaSuccess) {
    cudaGetLastError();
    return 0;
  }
  return n;
}

}  // namespace

int exec_packet_max_units_per_thread() { return kMaxUnitsPerThread; }
int exec_packet_max_threads() { return kMaxThreads; }

cudaError_t launch_exec_packet(int dtype, const PacketParams& P, int threads, bool overlap, cudaStream_t stream) {
  switch (dtype) {
    case PL_BF16: return launch_t<PL_BF16>(P, threads, overlap, stream);
    case PL_F32: return launch_t<PL_F32>(P, threads, overlap, stream);
    case PL_I32: return launch_t<PL_I32>(P, threads, overlap, stream);
    default: return cudaErrorInvalidValue;
  }
}

// how many rank groups (clusters of ctas_per_rank CTAs) can be resident at once
int exec_packet_max_groups(int dtype, int ctas_per_rank, int threads) {
  switch (dtype) {
    case PL_BF16: return clusters_t<PL_BF16>(ctas_per_rank, threads);
    case PL_F32: return clusters_t<PL_F32>(ctas_per_rank, threads);
    case PL_I32: return clusters_t<PL_I32>(ctas_per_rank, threads);
    default: return 0;
  }
}

}  // namespace pl
