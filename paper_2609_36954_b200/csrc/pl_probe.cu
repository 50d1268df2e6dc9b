// Diagnostic: what the bulk-copy machinery of the executors reaches on plain streams.
//
// Not part of the paper's method.  The roofline fractions of the collectives are quoted against
// a library copy; this probe measures, with the same instructions the executors use
// (cp.async.bulk global->shared with mbarrier completion, cp.async.bulk shared->global), the
// ceilings that bound them: a pure read (reduce-scatter and MoE combine are 8 reads to
// 1 write), a pure write, a copy, and one read to eight writes (all-gather and MoE dispatch).
//
// One warp per CTA, one CTA per SM (132 CTAs for the 1 : 8 stream), a ring of 6 tiles of 32 KiB.  CTA c handles tiles
// c, c + G, c + 2G, ...: at any moment the grid sweeps one compact window of the buffer.
#include <cuda_runtime.h>

#include <atomic>
#include <cstdint>

#include "pl_api_internal.h"
#include "pl_device.cuh"
#include "pl_internal.h"
#include "pl_ptx.cuh"
#include "purlin.h"

using namespace pl;

namespace {

constexpr uint32_t kTile = 32768;
constexpr uint32_t kSlots = 6;
constexpr size_t kSmem = 128 + (size_t)kSlots * kTile;
constexpr unsigned long long kLimitNs = 2000000000ull;

__device__ __forceinline__ unsigned long long now_ns() {
  unsigned long long t;
  asm volatile("mov.u64 %0, %globaltimer;" : "=l"(t));
  return t;
}

// bounded wait on a "tile landed" barrier; false when the time limit passed
__device__ __forceinline__ bool wait_full(uint64_t* bar, uint32_t parity) {
  if (ptx::mbar_try_wait(bar, parity)) return true;
  const unsigned long long t0 = now_ns();
  for (uint32_t tries = 1;; ++tries) {
    if (ptx::mbar_try_wait(bar, parity)) return true;
    if ((tries & 1023u) == 0 && now_ns() - t0 > kLimitNs) return false;
  }
}

// kind 0: read (tiles are loaded and dropped), 1: write (a fixed pattern tile is stored), 2: copy,
// 3: one read to eight writes (every tile is stored to the same offset of 8 consecutive regions of
// dst, each as long as src): the mix of the all-gather and of the MoE dispatch
// idle_count > 0: an SM-window launch (one CTA per SM; the CTAs on SMs idle_first .. idle_first +
// idle_count - 1 sit out, the others claim the n_active strides of the stream): see window_claim.
__device__ unsigned long long g_probe_window[3];

__global__ void __launch_bounds__(32) pl_probe_kernel(int kind, const char* src, char* dst, unsigned long long n_tiles,
                                                      int* status, int idle_first, int idle_count, int n_active) {
  extern __shared__ __align__(128) unsigned char smem[];
  uint64_t* full = reinterpret_cast<uint64_t*>(smem);
  unsigned char* tiles = smem + 128;
  const int lane = threadIdx.x;
  if (kind == 1) {
    // every tile carries the same non-constant pattern: 32-bit word j of a tile = j * 2654435761
    for (uint32_t i = lane; i < kSlots * kTile / 4; i += 32) reinterpret_cast<uint32_t*>(tiles)[i] = (i % (kTile / 4)) * 2654435761u;
    ptx::fence_proxy_async_smem();
  }
  if (lane == 0) {
    for (uint32_t s = 0; s < kSlots; ++s) ptx::mbar_init(full + s, 1);
    ptx::mbar_init_fence();
  }
  __syncwarp();
  if (lane != 0) return;
  unsigned long long c = blockIdx.x, G = gridDim.x;
  if (idle_count > 0) {
    uint32_t mask[5];
    for (int w = 0; w < 5; ++w) {
      mask[w] = 0xFFFFFFFFu;
      for (int b = 0; b < 32; ++b) {
        const int sm = w * 32 + b;
        if (sm >= idle_first && sm < idle_first + idle_count) mask[w] &= ~(1u << b);
      }
    }
    bool timed_out = false;
    const int slot = dev::window_claim(g_probe_window, mask, (uint32_t)n_active, kLimitNs, &timed_out);
    if (timed_out && status) *status = PL_ERR_TIMEOUT;
    if (slot < 0) {
      dev::window_leave(g_probe_window);
      return;
    }
    c = (unsigned long long)slot;
    G = (unsigned long long)n_active;
  }
  if (c >= n_tiles) {
    if (idle_count > 0) dev::window_leave(g_probe_window);
    return;
  }
  const unsigned long long n_my = (n_tiles - c + G - 1) / G;
  auto tile_off = [&](unsigned long long n) { return (c + n * G) * (unsigned long long)kTile; };
  unsigned long long issued = 0;  // loads issued so far (tiles 0 .. issued-1 of this CTA)
  auto load = [&](unsigned long long n) {
    const uint32_t s = (uint32_t)(n % kSlots);
    ptx::mbar_expect_tx(full + s, kTile);
    ptx::bulk_g2s(tiles + (size_t)s * kTile, src + tile_off(n), kTile, full + s);
    issued = n + 1;
  };
  bool ok = true;
  unsigned long long n = 0;
  if (kind != 1)
    for (unsigned long long k = 0; k < n_my && k < kSlots; ++k) load(k);
  for (; n < n_my; ++n) {
    const uint32_t s = (uint32_t)(n % kSlots), parity = (uint32_t)((n / kSlots) & 1);
    if (kind != 1 && !(ok = wait_full(full + s, parity))) break;
    if (kind == 0) {
      if (n + kSlots < n_my) load(n + kSlots);  // the tile is dropped: its slot is free at once
      continue;
    }
    if (kind == 3) {
      for (unsigned long long j = 0; j < 8; ++j)
        ptx::bulk_s2g(dst + j * n_tiles * kTile + tile_off(n), tiles + (size_t)s * kTile, kTile);
    } else {
      ptx::bulk_s2g(dst + tile_off(n), tiles + (size_t)s * kTile, kTile);
    }
    ptx::bulk_commit();
    if (kind >= 2 && n >= 2) {
      ptx::bulk_wait_read<2>();  // the store of tile n-2 no longer reads its slot
      if (n - 2 + kSlots < n_my) load(n - 2 + kSlots);
    } else if (kind == 1) {
      ptx::bulk_wait_read<8>();  // bounds the stores in flight; the pattern tiles are never rewritten
    }
  }
  ptx::bulk_wait<0>();
  if (!ok) {
    if (status) *status = PL_ERR_TIMEOUT;
    // loads already issued may still land: give each a bounded chance before leaving
    for (unsigned long long k = n; k < issued; ++k) {
      const uint32_t s = (uint32_t)(k % kSlots), parity = (uint32_t)((k / kSlots) & 1);
      for (uint32_t tries = 0; tries < (1u << 20) && !ptx::mbar_try_wait(full + s, parity); ++tries) {}
    }
  }
  if (idle_count > 0) dev::window_leave(g_probe_window);
}

}  // namespace

extern "C" pl_status_t pl_probe_hbm(int kind, const void* src, void* dst, size_t bytes, int32_t* status, void* stream) {
  if (kind < 0 || kind > 3 || bytes == 0 || bytes % kTile) return PL_ERR_INVALID_ARG;
  if ((kind != 1 && !src) || (kind != 0 && !dst)) return PL_ERR_INVALID_ARG;
  if (((uintptr_t)src & 15) || ((uintptr_t)dst & 15)) return PL_ERR_ALIGNMENT;
  int dev = 0, sms = 0;
  if (cudaGetDevice(&dev) != cudaSuccess || cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess) {
    cudaGetLastError();
    return PL_ERR_CUDA;
  }
  static std::atomic<unsigned long long> configured{0};  // shared-memory opt-in, one bit per device
  const unsigned long long bit = 1ull << (dev & 63);
  if (!(configured.load(std::memory_order_acquire) & bit)) {
    if (cudaFuncSetAttribute(pl_probe_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)kSmem) != cudaSuccess) {
      cudaGetLastError();
      return PL_ERR_CUDA;
    }
    configured.fetch_or(bit, std::memory_order_release);
  }
  cudaStream_t cs = static_cast<cudaStream_t>(stream);
  if (status && cudaMemsetAsync(status, 0, sizeof(int32_t), cs) != cudaSuccess) { cudaGetLastError(); return PL_ERR_CUDA; }
  // The write-dominated stream is fastest with about 8/9 of the SMs writing (132 of 148: 6.15-6.35 TB/s
  // against 5.7 TB/s with one CTA on every SM), and with the right ones sitting out: SMs 8-23 were a
  // good window on every B200 tried, the SMs a plain launch of 132 CTAs leaves idle only on some
  // (5.4 TB/s on the others).  The other streams want all SMs.  (Concurrent kind-3 probes on
  // different streams would share the window's claim words: the probe is a one-at-a-time tool.)
  const int active = kind == 3 ? ((sms * 8 / 9 + 3) & ~3) : sms;
  const bool window = kind == 3 && sms == 148 && active < sms;
  pl_probe_kernel<<<window ? sms : active, 32, kSmem, cs>>>(kind, static_cast<const char*>(src), static_cast<char*>(dst),
                                                             (unsigned long long)(bytes / kTile), reinterpret_cast<int*>(status),
                                                             8, window ? sms - active : 0, active);
  if (cudaGetLastError() != cudaSuccess) return PL_ERR_CUDA;
  g_launches.fetch_add(1);
  return PL_OK;
}
