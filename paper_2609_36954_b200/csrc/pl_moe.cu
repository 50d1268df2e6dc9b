// MoE expert-parallel dispatch / combine: an all-to-all-v of token rows whose counts are
// only known on the device (Table 2 of the paper names the pattern; Sec. 4 uses prefix sums
// for the variable-length offsets).
//
// dispatch = count (per 256-token block, per expert, via bit masks) -> scan (one CTA per
// source rank: exclusive prefix sums over its blocks, totals per expert and destination) ->
// place (segment bases in (source rank, expert, token) order, row index of every
// (token, slot), receive metadata) -> move (each token row is read once into
// shared memory by a bulk async copy and written to its K destinations by K bulk stores).
// combine = gate-weighted fp32 sum of the K expert rows of every token, ascending slot.
#include <cuda_bf16.h>
#include <cuda_runtime.h>

#include <atomic>
#include <cstring>
#include <new>
#include <vector>

#include "pl_api_internal.h"
#include "pl_internal.h"
#include "pl_ptx.cuh"

using namespace pl;

namespace {

constexpr int kTB = 256;             // tokens per count/place block
constexpr int kMaskWords = kTB / 32;
constexpr int kMaxTopk = 32;
constexpr uint32_t kMaxTile = 16384;  // bytes of a row moved per bulk copy

struct DispatchPtrs {
  const void* x[PL_MAX_RANKS];
  const int32_t* idx[PL_MAX_RANKS];
  void* recv[PL_MAX_RANKS];
  int32_t* meta[PL_MAX_RANKS];
};
struct CombinePtrs {
  const void* y[PL_MAX_RANKS];
  const float* gates[PL_MAX_RANKS];
  void* out[PL_MAX_RANKS];
};
struct MoeGeo {
  int R, T, E, K, NB, epr;
  uint32_t row_bytes, tile_bytes, n_tiles, slots;
  uint32_t rows_per_item, slot_bytes;  // mover: consecutive token rows per bulk load, bytes per ring slot
  unsigned long long cap;
  int32_t* blockcnt;   // [R][NB][E]: per-block counts, turned into exclusive block offsets by scan
  long long* counts;   // [R][R]
  long long* ecounts;  // [R][E]
  int32_t* pos;        // [R][T][K] row in the destination's receive buffer, -1 if dropped
  int32_t* prank;      // [R][T][K] destination rank
  int* flags;          // [0] overflow, [1] invalid expert id, [2] copy engine wait gave up, [3] grid barrier gave up (sticky)
  unsigned int* sync;  // fused bookkeeping: [0] CTAs that reached the grid barrier, [1] CTAs that left the kernel
  const int32_t* slotmask;  // optional [R][T][K]: written into the metadata instead of the slot index
  int gates_are_logits;     // combine: the gate input holds the K selected logits; softmax them first
};

__device__ __forceinline__ void build_mask(const MoeGeo& g, const int32_t* idx, uint32_t* mask, int t, int tid) {
  for (int i = tid; i < g.E * kMaskWords; i += kTB) mask[i] = 0u;
  __syncthreads();
  if (t < g.T)
    for (int j = 0; j < g.K; ++j) {
      const int e = idx[(size_t)t * g.K + j];
      if (e < 0) continue;  // empty slot (deduplicated routing pads with -1)
      if (e < g.E) atomicOr(&mask[e * kMaskWords + (tid >> 5)], 1u << (tid & 31));
      else g.flags[1] = 1;
    }
  __syncthreads();
}

__global__ void __launch_bounds__(kTB) moe_count_kernel(const __grid_constant__ DispatchPtrs P, const __grid_constant__ MoeGeo g) {
  extern __shared__ uint32_t mask[];
  const int b = blockIdx.x, p = blockIdx.y, tid = threadIdx.x;
  build_mask(g, P.idx[p], mask, b * kTB + tid, tid);
  for (int e = tid; e < g.E; e += kTB) {
    int c = 0;
#pragma unroll
    for (int w = 0; w < kMaskWords; ++w) c += __popc(mask[e * kMaskWords + w]);
    g.blockcnt[((size_t)p * g.NB + b) * g.E + e] = c;
  }
}

// One CTA per source rank p: exclusive scan of the per-block counts of every expert, the totals
// per expert (ecounts) and per destination rank (counts).  Segment bases, which need the counts
// of all source ranks, are computed by the place kernel.
__global__ void __launch_bounds__(256) moe_scan_kernel(const __grid_constant__ MoeGeo g) {
  const int tid = threadIdx.x, n = blockDim.x, p = blockIdx.x;
  if (p == 0 && tid < 3) g.flags[tid] = 0;
  for (int e = tid; e < g.E; e += n) {
    int run = 0;
    // exclusive scan over the token blocks, eight independent loads at a time
    for (int b0 = 0; b0 < g.NB; b0 += 8) {
      int v[8];
#pragma unroll
      for (int i = 0; i < 8; ++i)
        v[i] = (b0 + i < g.NB) ? g.blockcnt[((size_t)p * g.NB + b0 + i) * g.E + e] : 0;
#pragma unroll
      for (int i = 0; i < 8; ++i)
        if (b0 + i < g.NB) {
          g.blockcnt[((size_t)p * g.NB + b0 + i) * g.E + e] = run;
          run += v[i];
        }
    }
    g.ecounts[p * g.E + e] = run;
  }
  __syncthreads();  // this CTA's ecounts are visible to its own threads
  for (int r = tid; r < g.R; r += n) {
    long long s = 0;
    for (int e = r * g.epr; e < (r + 1) * g.epr; ++e) s += g.ecounts[p * g.E + e];
    g.counts[p * g.R + r] = s;
  }
}

__global__ void __launch_bounds__(kTB) moe_place_kernel(const __grid_constant__ DispatchPtrs P, const __grid_constant__ MoeGeo g) {
  extern __shared__ uint32_t mask[];
  int32_t* s_base = reinterpret_cast<int32_t*>(mask + (size_t)g.E * kMaskWords);  // [E] row of this source's segments
  const int b = blockIdx.x, p = blockIdx.y, tid = threadIdx.x, t = b * kTB + tid;
  const int32_t* idx = P.idx[p];
  // first row of expert e's run inside the receive buffer of its rank: everything sources
  // q < p send to that rank, then this source's rows for the rank's earlier experts
  for (int e = tid; e < g.E; e += kTB) {
    const int r = e / g.epr;
    long long off = 0;
    for (int q = 0; q < p; ++q) off += g.counts[q * g.R + r];
    for (int e2 = r * g.epr; e2 < e; ++e2) off += g.ecounts[p * g.E + e2];
    s_base[e] = (int32_t)off;
  }
  if (b == 0 && p == 0 && tid < g.R) {  // capacity check, once
    long long total = 0;
    for (int q = 0; q < g.R; ++q) total += g.counts[q * g.R + tid];
    if ((unsigned long long)total > g.cap) g.flags[0] = 1;
  }
  build_mask(g, idx, mask, t, tid);  // ends with a barrier: s_base is visible
  if (t >= g.T) return;
  const int w = tid >> 5;
  const uint32_t below = (1u << (tid & 31)) - 1u;
  for (int j = 0; j < g.K; ++j) {
    const int e = idx[(size_t)t * g.K + j];
    const size_t o = ((size_t)p * g.T + t) * g.K + j;
    if ((unsigned)e >= (unsigned)g.E) { g.pos[o] = -1; g.prank[o] = 0; continue; }
    int rank = __popc(mask[e * kMaskWords + w] & below);
    for (int w2 = 0; w2 < w; ++w2) rank += __popc(mask[e * kMaskWords + w2]);
    const long long row = (long long)s_base[e] + g.blockcnt[((size_t)p * g.NB + b) * g.E + e] + rank;
    const int r = e / g.epr;
    g.prank[o] = r;
    if ((unsigned long long)row < g.cap) {
      g.pos[o] = (int32_t)row;
      if (P.meta[r]) reinterpret_cast<int4*>(P.meta[r])[row] = make_int4(p, t, g.slotmask ? g.slotmask[o] : j, e);
    } else {
      g.pos[o] = -1;
    }
  }
}


// ---- fused bookkeeping: count -> (grid barrier) -> offsets -> place in ONE launch ------------
// Grid (NB, R), all CTAs co-resident (checked on the host).  Phase 1: the block's expert masks
// stay in shared memory and its per-expert counts go to global memory.  After a grid-wide
// barrier every CTA reads all R * NB * E counts (128 KiB at the C4 shape, from L2), derives the
// per-source totals, the segment bases of its own source rank and its own block offsets, and
// places its tokens.  The barrier is an arrival counter with a bounded wait; the last CTA to
// leave the kernel clears it, so nothing has to be reset between dispatches (or graph replays).
__global__ void __launch_bounds__(kTB) moe_plan_kernel(const __grid_constant__ DispatchPtrs P, const __grid_constant__ MoeGeo g) {
  extern __shared__ __align__(16) uint32_t mask[];
  int32_t* s_base = reinterpret_cast<int32_t*>(mask + (size_t)g.E * kMaskWords);  // [E]
  int32_t* s_ecnt = s_base + g.E;                                                 // [R][E] totals per (source, expert)
  int32_t* s_cnt = s_ecnt + (size_t)g.R * g.E;                                    // [R][R] rows source -> destination
  __shared__ int s_bad, s_giveup;
  const int b = blockIdx.x, p = blockIdx.y, tid = threadIdx.x, t = b * kTB + tid;
  const int32_t* idx = P.idx[p];
  asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
  if (tid == 0) { s_bad = 0; s_giveup = 0; }
  // ---- phase 1: masks and counts of this block
  for (int i = tid; i < g.E * kMaskWords; i += kTB) mask[i] = 0u;
  __syncthreads();
  if (t < g.T)
    for (int j0 = 0; j0 < g.K; j0 += 8) {
      int ev[8];  // eight slots at a time: the loads are independent of one another
#pragma unroll
      for (int k = 0; k < 8; ++k) ev[k] = (j0 + k < g.K) ? __ldg(&idx[(size_t)t * g.K + j0 + k]) : -1;
#pragma unroll
      for (int k = 0; k < 8; ++k) {
        const int e = ev[k];
        if (e < 0) continue;  // empty slot (deduplicated routing pads with -1)
        if (e < g.E) atomicOr(&mask[e * kMaskWords + (tid >> 5)], 1u << (tid & 31));
        else s_bad = 1;
      }
    }
  __syncthreads();
  for (int e = tid; e < g.E; e += kTB) {
    int c = 0;
#pragma unroll
    for (int w = 0; w < kMaskWords; ++w) c += __popc(mask[e * kMaskWords + w]);
    g.blockcnt[((size_t)p * g.NB + b) * g.E + e] = c;
  }
  if (b == 0 && p == 0 && tid < 3) g.flags[tid] = 0;  // ordered before every later flag write by the barrier
  // ---- grid barrier
  __syncthreads();
  if (tid == 0) {
    const unsigned int n_ctas = gridDim.x * gridDim.y;
    __threadfence();
    atomicAdd(g.sync, 1u);
    unsigned int seen;
    unsigned long long t0 = 0;
    uint32_t spins = 0;
    for (;;) {
      asm volatile("ld.acquire.gpu.global.u32 %0, [%1];" : "=r"(seen) : "l"(g.sync) : "memory");
      if (seen >= n_ctas) break;
      if ((++spins & 63u) == 0) {
        unsigned long long now;
        asm volatile("mov.u64 %0, %globaltimer;" : "=l"(now));
        if (t0 == 0) t0 = now;
        if (now - t0 > 2000000000ull) { s_giveup = 1; g.flags[3] = 1; break; }
      }
    }
  }
  __syncthreads();
  if (!s_giveup) {
    // ---- phase 2: totals per (source, expert); this block's offset inside its source's run.
    // Loads go out eight blocks at a time (independent, so one L2 latency per batch).
    if ((g.E & 3) == 0) {
      const int E4 = g.E >> 2;
      for (int i = tid; i < g.R * E4; i += kTB) {
        const int q = i / E4, e = (i - q * E4) << 2;
        int4 total = make_int4(0, 0, 0, 0), before = total;
        for (int b0 = 0; b0 < g.NB; b0 += 8) {
          int4 v[8];
#pragma unroll
          for (int k = 0; k < 8; ++k)
            v[k] = (b0 + k < g.NB) ? __ldcg(reinterpret_cast<const int4*>(&g.blockcnt[((size_t)q * g.NB + b0 + k) * g.E + e]))
                                   : make_int4(0, 0, 0, 0);
#pragma unroll
          for (int k = 0; k < 8; ++k) {
            if (b0 + k == b) before = total;
            total.x += v[k].x; total.y += v[k].y; total.z += v[k].z; total.w += v[k].w;
          }
        }
        *reinterpret_cast<int4*>(&s_ecnt[q * g.E + e]) = total;
        if (q == p) *reinterpret_cast<int4*>(&s_base[e]) = before;
      }
    } else {
      for (int i = tid; i < g.R * g.E; i += kTB) {
        const int q = i / g.E, e = i - q * g.E;
        int total = 0, before = 0;
        for (int b0 = 0; b0 < g.NB; b0 += 8) {
          int v[8];
#pragma unroll
          for (int k = 0; k < 8; ++k) v[k] = (b0 + k < g.NB) ? __ldcg(&g.blockcnt[((size_t)q * g.NB + b0 + k) * g.E + e]) : 0;
#pragma unroll
          for (int k = 0; k < 8; ++k) {
            if (b0 + k == b) before = total;
            total += v[k];
          }
        }
        s_ecnt[i] = total;
        if (q == p) s_base[e] = before;
      }
    }
    __syncthreads();
    for (int i = tid; i < g.R * g.R; i += kTB) {
      const int q = i / g.R, r = i - q * g.R;
      int c = 0;
      for (int e = r * g.epr; e < (r + 1) * g.epr; ++e) c += s_ecnt[q * g.E + e];
      s_cnt[i] = c;
    }
    __syncthreads();
    // first row of expert e's run in the receive buffer of its rank: what sources q < p send
    // there, then this source's rows for the rank's earlier experts, then the earlier blocks
    for (int e = tid; e < g.E; e += kTB) {
      const int r = e / g.epr;
      long long off = s_base[e];
      for (int q = 0; q < p; ++q) off += s_cnt[q * g.R + r];
      for (int e2 = r * g.epr; e2 < e; ++e2) off += s_ecnt[p * g.E + e2];
      s_base[e] = (int32_t)off;
      if (b == 0) g.ecounts[p * g.E + e] = s_ecnt[p * g.E + e];
    }
    if (b == 0 && tid < g.R) g.counts[p * g.R + tid] = s_cnt[p * g.R + tid];
    if (b == 0 && p == 0 && tid < g.R) {  // capacity check, once
      long long total = 0;
      for (int q = 0; q < g.R; ++q) total += s_cnt[q * g.R + tid];
      if ((unsigned long long)total > g.cap) g.flags[0] = 1;
    }
    if (tid == 0 && s_bad) g.flags[1] = 1;
    __syncthreads();
    // ---- phase 3: place this block's tokens
    if (t < g.T) {
      const int w = tid >> 5;
      const uint32_t below = (1u << (tid & 31)) - 1u;
      for (int j0 = 0; j0 < g.K; j0 += 8) {
        int ev[8];
#pragma unroll
        for (int k = 0; k < 8; ++k) ev[k] = (j0 + k < g.K) ? __ldg(&idx[(size_t)t * g.K + j0 + k]) : -1;
#pragma unroll
        for (int k = 0; k < 8; ++k) {
          const int j = j0 + k;
          if (j >= g.K) break;
          const int e = ev[k];
          const size_t o = ((size_t)p * g.T + t) * g.K + j;
          if ((unsigned)e >= (unsigned)g.E) { g.pos[o] = -1; g.prank[o] = 0; continue; }
          int rank = __popc(mask[e * kMaskWords + w] & below);
          for (int w2 = 0; w2 < w; ++w2) rank += __popc(mask[e * kMaskWords + w2]);
          const long long row = (long long)s_base[e] + rank;
          const int r = e / g.epr;
          g.prank[o] = r;
          if ((unsigned long long)row < g.cap) {
            g.pos[o] = (int32_t)row;
            if (P.meta[r]) reinterpret_cast<int4*>(P.meta[r])[row] = make_int4(p, t, g.slotmask ? g.slotmask[o] : j, e);
          } else {
            g.pos[o] = -1;
          }
        }
      }
    }
  }
  // ---- the last CTA to leave clears the barrier words for the next dispatch
  __syncthreads();
  if (tid == 0) {
    const unsigned int n_ctas = gridDim.x * gridDim.y;
    __threadfence();
    if (atomicAdd(g.sync + 1, 1u) == n_ctas - 1u) {
      g.sync[0] = 0u;
      g.sync[1] = 0u;
      __threadfence();
    }
  }
}

// Deduplicated routing: for every token the distinct destination ranks in ascending order
// (padded with -1) and, per destination, the mask of slots whose expert lives there.
__global__ void __launch_bounds__(256) moe_derive_ranks_kernel(const __grid_constant__ DispatchPtrs P, int R, int T, int K,
                                                               int epr, int KR, int32_t* ridx, int32_t* rmask) {
  const long long tok = (long long)blockIdx.x * blockDim.x + threadIdx.x;
  if (tok >= (long long)R * T) return;
  const int p = (int)(tok / T);
  const long long t = tok % T;
  const int32_t* idx = P.idx[p] + t * K;
  unsigned masks[PL_MAX_RANKS];
#pragma unroll
  for (int r = 0; r < PL_MAX_RANKS; ++r) masks[r] = 0u;
  for (int j = 0; j < K; ++j) {
    const int e = idx[j];
    const int r = (e >= 0) ? e / epr : -1;
#pragma unroll
    for (int q = 0; q < PL_MAX_RANKS; ++q)
      if (q == r) masks[q] |= 1u << j;
  }
  int n = 0;
#pragma unroll
  for (int r = 0; r < PL_MAX_RANKS; ++r)
    if (r < R && masks[r]) {
      ridx[tok * KR + n] = r;
      rmask[tok * KR + n] = (int32_t)masks[r];
      ++n;
    }
  for (; n < KR; ++n) {
    ridx[tok * KR + n] = -1;
    rmask[tok * KR + n] = 0;
  }
}

// One warp per CTA drives a ring of `slots` shared-memory tiles: lane 0 issues the bulk loads
// (prime, then refill as tiles drain: the paper's Algorithm 2 with the processing step being
// "store to K places"), the lanes share the bulk stores.  A work item is a group of `rows`
// consecutive token rows of one source rank, which are contiguous in its input: one bulk load of
// up to 56 KiB, then rows x K bulk stores of one row each (rows wider than 16 KiB are moved in
// tiles, one row per item).  The write-dominated stream this kernel is runs fastest with large
// loads and 128-136 CTAs on this GPU (1 read : 8 writes through the same ring: 6.15-6.3 TB/s with
// 128-136 CTAs and 32-64 KiB tiles, 5.65-5.73 TB/s with 140-148 CTAs, 5.55 TB/s with 296 CTAs and
// 14 KiB tiles), so the grid is a property of the GPU's memory system, not of the row count.
__global__ void __launch_bounds__(32) moe_move_kernel(const __grid_constant__ DispatchPtrs P, const __grid_constant__ MoeGeo g) {
  extern __shared__ __align__(128) unsigned char smem[];
  const int lane = threadIdx.x;
  const uint32_t S = g.slots;
  uint64_t* full = reinterpret_cast<uint64_t*>(smem);
  unsigned char* tiles = smem + 128;
  if (lane == 0) {
    for (uint32_t s = 0; s < S; ++s) ptx::mbar_init(full + s, 1);
    ptx::mbar_init_fence();
  }
  __syncwarp();
  // launched with programmatic stream serialization: set up above while the bookkeeping kernel
  // drains, wait here for it to complete before anything it wrote (pos, prank) is read
  asm volatile("griddepcontrol.wait;" ::: "memory");
  const uint32_t rows = g.rows_per_item;  // > 1 only when a row is one tile
  const unsigned long long groups_per_rank = ((unsigned long long)g.T + rows - 1) / rows;
  const unsigned long long n_items = (unsigned long long)g.R * groups_per_rank * g.n_tiles;
  const unsigned long long c = blockIdx.x, G = gridDim.x;
  if (c >= n_items) return;
  const unsigned long long n_my = (n_items - c + G - 1) / G;
  constexpr int L = 2;  // store groups allowed to be still reading shared memory

  // item n of this CTA: tokens [tok, tok + nrows) of one rank, bytes [off, off + bytes) of each row
  auto item = [&](unsigned long long n, unsigned long long& tok, uint32_t& nrows, uint32_t& off, uint32_t& bytes) {
    const unsigned long long w = c + n * G;
    const unsigned long long grp = w / g.n_tiles;
    const uint32_t tile = (uint32_t)(w % g.n_tiles);
    const unsigned long long p = grp / groups_per_rank, t0 = (grp % groups_per_rank) * rows;
    tok = p * g.T + t0;
    nrows = (uint32_t)min((unsigned long long)rows, (unsigned long long)g.T - t0);
    off = tile * g.tile_bytes;
    bytes = (rows > 1) ? g.row_bytes : min(g.tile_bytes, g.row_bytes - off);
  };
  auto issue_load = [&](unsigned long long n) {
    unsigned long long tok;
    uint32_t nrows, off, bytes;
    item(n, tok, nrows, off, bytes);
    const int p = (int)(tok / g.T);
    const unsigned long long t = tok % g.T;
    const char* src = static_cast<const char*>(P.x[p]) + t * g.row_bytes + off;
    const uint32_t s = (uint32_t)(n % S);
    ptx::mbar_expect_tx(full + s, nrows * bytes);
    ptx::bulk_g2s_hint(tiles + (size_t)s * g.slot_bytes, src, nrows * bytes, full + s, ptx::policy_evict_first());
  };

  unsigned long long issued = 0;
  if (lane == 0)
    for (; issued < n_my && issued < S; ++issued) issue_load(issued);
  issued = min(n_my, (unsigned long long)S);
  bool failed = false;
  unsigned long long n = 0;
  for (; n < n_my; ++n) {
    unsigned long long tok;
    uint32_t nrows, off, bytes;
    item(n, tok, nrows, off, bytes);
    // this lane's first store of the item: (row i of the group, slot j); fetched before the wait
    const uint32_t n_st = nrows * (uint32_t)g.K;
    int row = -1, r = 0;
    if ((uint32_t)lane < n_st) {
      row = g.pos[tok * g.K + lane];
      r = g.prank[tok * g.K + lane];
    }
    const uint32_t s = (uint32_t)(n % S), parity = (uint32_t)((n / S) & 1);
    // bounded wait for the tile to land
    bool ok = ptx::mbar_try_wait(full + s, parity);
    if (!ok) {
      unsigned long long t0 = 0;
      asm volatile("mov.u64 %0, %globaltimer;" : "=l"(t0));
      for (uint32_t tries = 1; !(ok = ptx::mbar_try_wait(full + s, parity)); ++tries) {
        if ((tries & 1023u) == 0) {
          unsigned long long t1;
          asm volatile("mov.u64 %0, %globaltimer;" : "=l"(t1));
          if (t1 - t0 > 2000000000ull) break;
        }
      }
    }
    ok = __all_sync(0xFFFFFFFFu, ok);
    if (!ok) { failed = true; break; }
    // every token row is read once and every received row written once: both stream through L2
    const unsigned char* tile = tiles + (size_t)s * g.slot_bytes;
    for (uint32_t idx = lane; idx < n_st; idx += 32) {
      if (idx >= 32) {
        row = g.pos[tok * g.K + idx];
        r = g.prank[tok * g.K + idx];
      }
      if (row >= 0)
        ptx::bulk_s2g_hint(static_cast<char*>(P.recv[r]) + (size_t)row * g.row_bytes + off,
                           tile + (size_t)(idx / (uint32_t)g.K) * bytes, bytes, ptx::policy_evict_first());
    }
    ptx::bulk_commit();
    if (n >= (unsigned long long)L) {
      ptx::bulk_wait_read<L>();
      __syncwarp();
      const unsigned long long m = n - L;  // its tile is no longer being read
      if (lane == 0 && m + S < n_my) issue_load(m + S);
    }
  }
  ptx::bulk_wait<0>();
  if (failed && lane == 0) {
    g.flags[2] = 1;
    // loads already issued may still land: give each a bounded chance before leaving
    const unsigned long long last = min(n_my, n + S);
    for (unsigned long long k = n; k < last; ++k) {
      const uint32_t s = (uint32_t)(k % S), parity = (uint32_t)((k / S) & 1);
      for (uint32_t tries = 0; tries < (1u << 20) && !ptx::mbar_try_wait(full + s, parity); ++tries) {}
    }
  }
}

// combine: CTA per token (grid-strided), 16-byte column units across threads, the K source
// rows and gates of the next token are fetched while the current one is summed.
constexpr int kCombineThreads = 256;
__global__ void __launch_bounds__(kCombineThreads) moe_combine_kernel(const __grid_constant__ CombinePtrs P, const __grid_constant__ MoeGeo g) {
  __shared__ const char* s_row[2][kMaxTopk];
  __shared__ float s_gate[2][kMaxTopk];
  const int tid = threadIdx.x;
  const unsigned long long n_tok = (unsigned long long)g.R * g.T;
  auto load_meta = [&](unsigned long long tok, int buf) {
    if (tid < g.K) {
      const int p = (int)(tok / g.T);
      const unsigned long long t = tok % g.T;
      const int row = g.pos[tok * g.K + tid];
      const int r = g.prank[tok * g.K + tid];
      s_row[buf][tid] = row >= 0 ? static_cast<const char*>(P.y[r]) + (size_t)row * g.row_bytes : nullptr;
      float gate = P.gates[p][t * g.K + tid];
      if (g.gates_are_logits) {
        // fp32 softmax over the token's K logits (max-subtracted); K <= 32 lanes of warp 0
        const unsigned lanes = (g.K >= 32) ? 0xFFFFFFFFu : ((1u << g.K) - 1u);
        float m = gate;
        for (int j = 0; j < g.K; ++j) m = fmaxf(m, __shfl_sync(lanes, gate, j));
        const float e = expf(gate - m);
        float sum = 0.f;
        for (int j = 0; j < g.K; ++j) sum += __shfl_sync(lanes, e, j);  // ascending slot order on every lane
        gate = e / sum;
      }
      s_gate[buf][tid] = gate;
    }
  };
  unsigned long long tok = blockIdx.x;
  if (tok < n_tok) load_meta(tok, 0);
  __syncthreads();
  const uint32_t units = g.row_bytes >> 4;
  for (int it = 0; tok < n_tok; tok += gridDim.x, ++it) {
    const int buf = it & 1;
    if (tok + gridDim.x < n_tok) load_meta(tok + gridDim.x, buf ^ 1);
    const int p = (int)(tok / g.T);
    char* out = static_cast<char*>(P.out[p]) + (tok % g.T) * g.row_bytes;
    for (uint32_t u = tid; u < units; u += kCombineThreads) {
      float acc[8];
#pragma unroll
      for (int i = 0; i < 8; ++i) acc[i] = 0.f;
      for (int j0 = 0; j0 < g.K; j0 += 8) {
        uint4 q[8];
#pragma unroll
        for (int j = 0; j < 8; ++j) {
          const char* rowp = (j0 + j < g.K) ? s_row[buf][j0 + j] : nullptr;
          q[j] = rowp ? __ldcg(reinterpret_cast<const uint4*>(rowp) + u) : make_uint4(0, 0, 0, 0);
        }
#pragma unroll
        for (int j = 0; j < 8; ++j) {
          if (j0 + j < g.K) {
            const float gt = s_gate[buf][j0 + j];
            const uint32_t w[4] = {q[j].x, q[j].y, q[j].z, q[j].w};
#pragma unroll
            for (int i = 0; i < 4; ++i) {
              acc[2 * i] = fmaf(gt, __uint_as_float(w[i] << 16), acc[2 * i]);
              acc[2 * i + 1] = fmaf(gt, __uint_as_float(w[i] & 0xFFFF0000u), acc[2 * i + 1]);
            }
          }
        }
      }
      uint4 o;
      __nv_bfloat162 a = __floats2bfloat162_rn(acc[0], acc[1]);
      __nv_bfloat162 b = __floats2bfloat162_rn(acc[2], acc[3]);
      __nv_bfloat162 c2 = __floats2bfloat162_rn(acc[4], acc[5]);
      __nv_bfloat162 d = __floats2bfloat162_rn(acc[6], acc[7]);
      o.x = *reinterpret_cast<uint32_t*>(&a);
      o.y = *reinterpret_cast<uint32_t*>(&b);
      o.z = *reinterpret_cast<uint32_t*>(&c2);
      o.w = *reinterpret_cast<uint32_t*>(&d);
      __stcg(reinterpret_cast<uint4*>(out) + u, o);
    }
    __syncthreads();
  }
}

size_t align_up(size_t x, size_t a) { return (x + a - 1) / a * a; }

// The dynamic shared-memory limit is an attribute of the FUNCTION (per device), not of a plan:
// it is raised once per device to the most any plan can ask for, so that creating a second,
// smaller plan cannot lower it under the feet of the first.
constexpr int kMaxExperts = 4096;
constexpr size_t kMoveSmemMax = 227 * 1024;
constexpr size_t kPlanSmemMax = 200 * 1024;  // the fused bookkeeping kernel is used while its tables fit this

size_t plan_smem_bytes(const MoeGeo& g) {
  return ((size_t)g.E * kMaskWords + (size_t)g.E + (size_t)g.R * g.E + (size_t)g.R * g.R) * 4;
}
bool configure_kernels(int device) {
  static std::atomic<unsigned long long> configured{0};
  const unsigned long long bit = 1ull << (device & 63);
  if (configured.load(std::memory_order_acquire) & bit) return true;
  if (cudaFuncSetAttribute(moe_move_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)kMoveSmemMax) != cudaSuccess ||
      cudaFuncSetAttribute(moe_count_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, kMaxExperts * kMaskWords * 4) != cudaSuccess ||
      cudaFuncSetAttribute(moe_place_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, kMaxExperts * kMaskWords * 4 + kMaxExperts * 4) != cudaSuccess ||
      cudaFuncSetAttribute(moe_plan_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)kPlanSmemMax) != cudaSuccess) {
    cudaGetLastError();
    return false;
  }
  configured.fetch_or(bit, std::memory_order_release);
  return true;
}

}  // namespace

struct pl_moe_plan_s {
  pl_comm_t comm = nullptr;
  MoeGeo g{};
  char* d_blob = nullptr;
  size_t blob_bytes = 0;
  int sm_count = 148;
  int combine_per_sm = 4;  // resident CTAs of the combine kernel per SM (occupancy query at plan creation)
  size_t move_smem = 0;
  bool fused = false, fused_dedup = false;  // bookkeeping in one launch (grid co-resident, tables fit shared memory)
  bool dispatched = false;
  // deduplicated variant: the same machinery run over "one expert per rank" routing
  MoeGeo gd{};
  int32_t* d_ridx = nullptr;   // [R][T][KR] distinct destination ranks, -1 padded
  int32_t* d_rmask = nullptr;  // [R][T][KR] slot masks
  float* d_ones = nullptr;     // [T][KR] unit gates
  char* d_blob2 = nullptr;
  bool dispatched_dedup = false;
};

extern "C" {

pl_status_t pl_moe_plan_create(pl_comm_t comm, int tokens_per_rank, int hidden, int n_experts, int topk,
                               size_t recv_capacity_rows, pl_moe_plan_t* out) {
  if (!comm || !out) return PL_ERR_INVALID_ARG;
  *out = nullptr;
  if (comm->planner) return PL_ERR_UNSUPPORTED;
  if (!on_comm_device(comm)) return PL_ERR_INVALID_ARG;
  const int R = comm->R;
  if (tokens_per_rank < 1 || hidden < 1 || n_experts < R || topk < 1 || topk > kMaxTopk) return PL_ERR_INVALID_ARG;
  if (n_experts % R || n_experts > kMaxExperts || topk > n_experts) return PL_ERR_INVALID_ARG;
  if (recv_capacity_rows == 0 || recv_capacity_rows > 0x7FFFFFFFull) return PL_ERR_INVALID_ARG;
  const size_t row_bytes = (size_t)hidden * elem_size(comm->dtype);
  if (row_bytes % 16) return PL_ERR_ALIGNMENT;
  if (row_bytes > (1u << 30)) return PL_ERR_INVALID_ARG;
  pl_moe_plan_s* pl = new (std::nothrow) pl_moe_plan_s();
  if (!pl) return PL_ERR_OOM;
  pl->comm = comm;
  pl->sm_count = comm->sm_count;
  {
    // The combine kernel deals tokens to CTAs by a fixed stride, so its grid must be exactly one
    // resident wave: with 1.5 waves (6 CTAs per SM against 4 resident) the second half wave ran
    // alone and the launch took 703 us instead of 612 us (C4 shape).
    int occ = 0;
    if (cudaOccupancyMaxActiveBlocksPerMultiprocessor(&occ, moe_combine_kernel, kCombineThreads, 0) != cudaSuccess || occ < 1) {
      cudaGetLastError();
      occ = 1;
    }
    pl->combine_per_sm = occ;
  }
  MoeGeo& g = pl->g;
  g.R = R;
  g.T = tokens_per_rank;
  g.E = n_experts;
  g.K = topk;
  g.NB = (tokens_per_rank + kTB - 1) / kTB;
  g.epr = n_experts / R;
  g.row_bytes = (uint32_t)row_bytes;
  g.n_tiles = (uint32_t)((row_bytes + kMaxTile - 1) / kMaxTile);
  g.tile_bytes = (uint32_t)align_up((row_bytes + g.n_tiles - 1) / g.n_tiles, 16);
  // Rows of at most one tile are moved in groups of consecutive tokens, up to 56 KiB per bulk load,
  // through exactly three slots: two store groups may still read their tiles while the third tile
  // is loaded.  Measured at the C4 shape (14,336-byte rows, 8 stores per row): 4 rows x 3 slots
  // 722-726 us; 4 slots 787 us, 2 or 3 rows per load with 4-6 slots 785-793 us, one row per load
  // 771 us: the write-dominated stream wants large loads and few bytes in flight.  Wider rows go
  // tile by tile through at least 4 slots.
  g.rows_per_item = g.n_tiles == 1 ? (uint32_t)std::max<size_t>(1, std::min<size_t>(32, 57344 / g.tile_bytes)) : 1u;
  g.slot_bytes = g.rows_per_item * g.tile_bytes;
  g.slots = g.rows_per_item > 1 ? 3u : (uint32_t)std::min<size_t>(8, std::max<size_t>(4, (96 * 1024) / g.tile_bytes));
  g.cap = recv_capacity_rows;
  pl->move_smem = 128 + (size_t)g.slots * g.slot_bytes;
  size_t off = 0;
  auto place = [&](size_t bytes) { size_t o = off; off = align_up(off + bytes, 256); return o; };
  const size_t o_bc = place((size_t)R * g.NB * g.E * 4);
  const size_t o_cnt = place((size_t)R * R * 8), o_ecnt = place((size_t)R * g.E * 8);
  const size_t o_pos = place((size_t)R * g.T * g.K * 4), o_prank = place((size_t)R * g.T * g.K * 4);
  const size_t o_flags = place(32);  // 4 flag words + 2 barrier words
  pl->blob_bytes = off;
  if (cudaMalloc(&pl->d_blob, off) != cudaSuccess) { cudaGetLastError(); delete pl; return PL_ERR_OOM; }
  if (cudaMemset(pl->d_blob, 0, off) != cudaSuccess) { cudaGetLastError(); cudaFree(pl->d_blob); delete pl; return PL_ERR_CUDA; }
  g.blockcnt = reinterpret_cast<int32_t*>(pl->d_blob + o_bc);
  g.counts = reinterpret_cast<long long*>(pl->d_blob + o_cnt);
  g.ecounts = reinterpret_cast<long long*>(pl->d_blob + o_ecnt);
  g.pos = reinterpret_cast<int32_t*>(pl->d_blob + o_pos);
  g.prank = reinterpret_cast<int32_t*>(pl->d_blob + o_prank);
  g.flags = reinterpret_cast<int*>(pl->d_blob + o_flags);
  g.sync = reinterpret_cast<unsigned int*>(pl->d_blob + o_flags + 16);
  if (!configure_kernels(comm->device)) {
    cudaFree(pl->d_blob);
    delete pl;
    return PL_ERR_CUDA;
  }
  // second set of bookkeeping for the deduplicated variant: R "experts" (one per rank),
  // at most min(topk, R) destinations per token
  {
    MoeGeo& d = pl->gd;
    d = g;
    d.E = R;
    d.epr = 1;
    d.K = std::min(topk, R);
    size_t off2 = 0;
    auto place2 = [&](size_t bytes) { size_t o = off2; off2 = align_up(off2 + bytes, 256); return o; };
    const size_t tk = (size_t)R * g.T * d.K;
    const size_t q_bc = place2((size_t)R * g.NB * R * 4);
    const size_t q_cnt = place2((size_t)R * R * 8), q_ecnt = place2((size_t)R * R * 8);
    const size_t q_pos = place2(tk * 4), q_prank = place2(tk * 4), q_ridx = place2(tk * 4), q_rmask = place2(tk * 4);
    const size_t q_ones = place2((size_t)g.T * d.K * 4), q_flags = place2(32);
    if (cudaMalloc(&pl->d_blob2, off2) != cudaSuccess) { cudaGetLastError(); cudaFree(pl->d_blob); delete pl; return PL_ERR_OOM; }
    std::vector<float> ones((size_t)g.T * d.K, 1.0f);
    if (cudaMemset(pl->d_blob2, 0, off2) != cudaSuccess ||
        cudaMemcpy(pl->d_blob2 + q_ones, ones.data(), ones.size() * 4, cudaMemcpyHostToDevice) != cudaSuccess) {
      cudaGetLastError();
      cudaFree(pl->d_blob);
      cudaFree(pl->d_blob2);
      delete pl;
      return PL_ERR_CUDA;
    }
    d.blockcnt = reinterpret_cast<int32_t*>(pl->d_blob2 + q_bc);
    d.counts = reinterpret_cast<long long*>(pl->d_blob2 + q_cnt);
    d.ecounts = reinterpret_cast<long long*>(pl->d_blob2 + q_ecnt);
    d.pos = reinterpret_cast<int32_t*>(pl->d_blob2 + q_pos);
    d.prank = reinterpret_cast<int32_t*>(pl->d_blob2 + q_prank);
    d.flags = reinterpret_cast<int*>(pl->d_blob2 + q_flags);
    d.sync = reinterpret_cast<unsigned int*>(pl->d_blob2 + q_flags + 16);
    pl->d_ridx = reinterpret_cast<int32_t*>(pl->d_blob2 + q_ridx);
    pl->d_rmask = reinterpret_cast<int32_t*>(pl->d_blob2 + q_rmask);
    pl->d_ones = reinterpret_cast<float*>(pl->d_blob2 + q_ones);
    d.slotmask = pl->d_rmask;
  }
  {
    // one-launch bookkeeping needs every CTA of its grid resident at once (they meet at a barrier)
    auto feasible = [&](const MoeGeo& q) {
      const size_t smem = plan_smem_bytes(q);
      if (smem > kPlanSmemMax) return false;
      int per_sm = 0;
      if (cudaOccupancyMaxActiveBlocksPerMultiprocessor(&per_sm, moe_plan_kernel, kTB, smem) != cudaSuccess) {
        cudaGetLastError();
        return false;
      }
      return (long long)q.NB * q.R <= (long long)per_sm * comm->sm_count;
    };
    pl->fused = feasible(pl->g);
    pl->fused_dedup = feasible(pl->gd);
  }
  comm->n_plans += 1;
  *out = pl;
  return PL_OK;
}

pl_status_t pl_moe_plan_destroy(pl_moe_plan_t plan) {
  if (!plan) return PL_ERR_INVALID_ARG;
  if (plan->d_blob) cudaFree(plan->d_blob);
  if (plan->d_blob2) cudaFree(plan->d_blob2);
  plan->comm->n_plans -= 1;
  delete plan;
  return PL_OK;
}

// count / scan / place (or the fused kernel), then the row mover launched so that its set-up
// overlaps the tail of the bookkeeping.  Returns the number of kernels launched, 0 on error.
static int launch_dispatch(pl_moe_plan_t plan, const DispatchPtrs& P, const MoeGeo& g, bool fused, cudaStream_t cs) {
  int launched = 0;
  const size_t mask_smem = (size_t)g.E * kMaskWords * 4;
  dim3 grid(g.NB, g.R);
  if (fused) {
    moe_plan_kernel<<<grid, kTB, plan_smem_bytes(g), cs>>>(P, g);
    launched = 1;
  } else {
    moe_count_kernel<<<grid, kTB, mask_smem, cs>>>(P, g);
    moe_scan_kernel<<<g.R, 256, 0, cs>>>(g);
    moe_place_kernel<<<grid, kTB, mask_smem + (size_t)g.E * 4, cs>>>(P, g);
    launched = 3;
  }
  if (cudaGetLastError() != cudaSuccess) return 0;
  const unsigned long long items = (unsigned long long)g.R * ((g.T + g.rows_per_item - 1) / g.rows_per_item) * g.n_tiles;
  const int per_sm = (int)std::max<size_t>(1, std::min<size_t>(4, (227 * 1024) / plan->move_smem));
  int mgrid = (int)std::min<unsigned long long>(items, (unsigned long long)plan->sm_count * per_sm);
  // Grouped rows: about 8/9 of the SMs, one CTA each (132 on a B200).  The 1 read : K writes stream
  // is fastest there: 722-726 us at the C4 shape with 128-132 CTAs, 734-744 us with 136-148, 737 us
  // with 296 (two per SM), 749-794 us with 112-120.
  if (g.rows_per_item > 1) mgrid = (int)std::min<unsigned long long>(items, (unsigned long long)((plan->sm_count * 8 / 9 + 3) & ~3));
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = dim3((unsigned)mgrid);
  cfg.blockDim = dim3(32);
  cfg.dynamicSmemBytes = plan->move_smem;
  cfg.stream = cs;
  cudaLaunchAttribute attr[1];
  attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  attr[0].val.programmaticStreamSerializationAllowed = 1;
  cfg.attrs = attr;
  cfg.numAttrs = fused ? 1 : 0;  // only the fused kernel releases its dependents early
  if (cudaLaunchKernelEx(&cfg, moe_move_kernel, P, g) != cudaSuccess) { cudaGetLastError(); return 0; }
  return launched + 1;
}

pl_status_t pl_moe_dispatch(pl_moe_plan_t plan, const void* const* x, const int32_t* const* topk_idx,
                            void* const* recv, int32_t* const* recv_meta, void* stream) {
  if (!plan || !x || !topk_idx || !recv) return PL_ERR_INVALID_ARG;
  if (!on_comm_device(plan->comm)) return PL_ERR_INVALID_ARG;
  const MoeGeo& g = plan->g;
  DispatchPtrs P;
  std::memset(&P, 0, sizeof(P));
  for (int r = 0; r < g.R; ++r) {
    if (!x[r] || !topk_idx[r] || !recv[r]) return PL_ERR_INVALID_ARG;
    if (((uintptr_t)x[r] & 15) || ((uintptr_t)recv[r] & 15) || ((uintptr_t)topk_idx[r] & 3)) return PL_ERR_ALIGNMENT;
    if (recv_meta && recv_meta[r] && ((uintptr_t)recv_meta[r] & 15)) return PL_ERR_ALIGNMENT;
    P.x[r] = x[r];
    P.idx[r] = topk_idx[r];
    P.recv[r] = recv[r];
    P.meta[r] = recv_meta ? recv_meta[r] : nullptr;
  }
  const int launched = launch_dispatch(plan, P, g, plan->fused, static_cast<cudaStream_t>(stream));
  if (!launched) return PL_ERR_CUDA;
  g_launches.fetch_add(launched);
  plan->dispatched = true;
  return PL_OK;
}

static pl_status_t combine_impl(pl_moe_plan_t plan, const void* const* y, const float* const* gates, void* const* out,
                                void* stream, bool gates_are_logits) {
  if (!plan || !y || !gates || !out) return PL_ERR_INVALID_ARG;
  if (plan->comm->dtype != PL_BF16) return PL_ERR_UNSUPPORTED;
  if (!plan->dispatched) return PL_ERR_INVALID_ARG;
  if (!on_comm_device(plan->comm)) return PL_ERR_INVALID_ARG;
  MoeGeo g = plan->g;  // by value: the mode below belongs to this call, not to the plan
  g.gates_are_logits = gates_are_logits ? 1 : 0;
  CombinePtrs P;
  std::memset(&P, 0, sizeof(P));
  for (int r = 0; r < g.R; ++r) {
    if (!y[r] || !gates[r] || !out[r]) return PL_ERR_INVALID_ARG;
    if (((uintptr_t)y[r] & 15) || ((uintptr_t)out[r] & 15) || ((uintptr_t)gates[r] & 3)) return PL_ERR_ALIGNMENT;
    P.y[r] = y[r];
    P.gates[r] = gates[r];
    P.out[r] = out[r];
  }
  const unsigned long long n_tok = (unsigned long long)g.R * g.T;
  const int grid = (int)std::min<unsigned long long>(n_tok, (unsigned long long)plan->sm_count * plan->combine_per_sm);
  moe_combine_kernel<<<grid, kCombineThreads, 0, static_cast<cudaStream_t>(stream)>>>(P, g);
  if (cudaGetLastError() != cudaSuccess) return PL_ERR_CUDA;
  g_launches.fetch_add(1);
  return PL_OK;
}

pl_status_t pl_moe_combine(pl_moe_plan_t plan, const void* const* y, const float* const* gates, void* const* out,
                           void* stream) {
  return combine_impl(plan, y, gates, out, stream, false);
}

pl_status_t pl_moe_combine_logits(pl_moe_plan_t plan, const void* const* y, const float* const* logits,
                                  void* const* out, void* stream) {
  return combine_impl(plan, y, logits, out, stream, true);
}

pl_status_t pl_moe_plan_read(pl_moe_plan_t plan, int32_t* pos, int64_t* counts, int64_t* expert_counts, void* stream) {
  if (!plan) return PL_ERR_INVALID_ARG;
  const MoeGeo& g = plan->g;
  if (cudaStreamSynchronize(static_cast<cudaStream_t>(stream)) != cudaSuccess) { cudaGetLastError(); return PL_ERR_CUDA; }
  int flags[4] = {0, 0, 0, 0};
  bool ok = cudaMemcpy(flags, g.flags, 16, cudaMemcpyDeviceToHost) == cudaSuccess;
  if (ok && flags[3]) {  // the grid barrier of the bookkeeping kernel gave up: report once, clear barrier state
    flags[2] = 1;
    ok = cudaMemset(g.flags + 3, 0, 4 + 8) == cudaSuccess;  // flags[3] and the two barrier words behind it
  }
  if (ok && pos) ok = cudaMemcpy(pos, g.pos, (size_t)g.R * g.T * g.K * 4, cudaMemcpyDeviceToHost) == cudaSuccess;
  if (ok && counts) ok = cudaMemcpy(counts, g.counts, (size_t)g.R * g.R * 8, cudaMemcpyDeviceToHost) == cudaSuccess;
  if (ok && expert_counts) ok = cudaMemcpy(expert_counts, g.ecounts, (size_t)g.R * g.E * 8, cudaMemcpyDeviceToHost) == cudaSuccess;
  if (!ok) { cudaGetLastError(); return PL_ERR_CUDA; }
  if (flags[2]) return PL_ERR_TIMEOUT;
  if (flags[1]) return PL_ERR_INVALID_ARG;
  if (flags[0]) return PL_ERR_OVERFLOW;
  return PL_OK;
}

pl_status_t pl_moe_dispatch_dedup(pl_moe_plan_t plan, const void* const* x, const int32_t* const* topk_idx,
                                  void* const* recv, int32_t* const* recv_meta, void* stream) {
  if (!plan || !x || !topk_idx || !recv) return PL_ERR_INVALID_ARG;
  if (!on_comm_device(plan->comm)) return PL_ERR_INVALID_ARG;
  const MoeGeo& g = plan->g;
  const MoeGeo& d = plan->gd;
  DispatchPtrs P0, P;
  std::memset(&P0, 0, sizeof(P0));
  std::memset(&P, 0, sizeof(P));
  for (int r = 0; r < g.R; ++r) {
    if (!x[r] || !topk_idx[r] || !recv[r]) return PL_ERR_INVALID_ARG;
    if (((uintptr_t)x[r] & 15) || ((uintptr_t)recv[r] & 15) || ((uintptr_t)topk_idx[r] & 3)) return PL_ERR_ALIGNMENT;
    if (recv_meta && recv_meta[r] && ((uintptr_t)recv_meta[r] & 15)) return PL_ERR_ALIGNMENT;
    P0.idx[r] = topk_idx[r];
    P.x[r] = x[r];
    P.idx[r] = plan->d_ridx + (size_t)r * g.T * d.K;  // the derived per-rank routing
    P.recv[r] = recv[r];
    P.meta[r] = recv_meta ? recv_meta[r] : nullptr;
  }
  cudaStream_t cs = static_cast<cudaStream_t>(stream);
  const long long n_tok = (long long)g.R * g.T;
  moe_derive_ranks_kernel<<<(unsigned)((n_tok + 255) / 256), 256, 0, cs>>>(P0, g.R, g.T, g.K, g.epr, d.K, plan->d_ridx, plan->d_rmask);
  if (cudaGetLastError() != cudaSuccess) return PL_ERR_CUDA;
  const int launched = launch_dispatch(plan, P, d, plan->fused_dedup, cs);
  if (!launched) return PL_ERR_CUDA;
  g_launches.fetch_add(1 + launched);
  plan->dispatched_dedup = true;
  return PL_OK;
}

pl_status_t pl_moe_combine_dedup(pl_moe_plan_t plan, const void* const* z, void* const* out, void* stream) {
  if (!plan || !z || !out) return PL_ERR_INVALID_ARG;
  if (plan->comm->dtype != PL_BF16) return PL_ERR_UNSUPPORTED;
  if (!plan->dispatched_dedup) return PL_ERR_INVALID_ARG;
  if (!on_comm_device(plan->comm)) return PL_ERR_INVALID_ARG;
  const MoeGeo& d = plan->gd;
  CombinePtrs P;
  std::memset(&P, 0, sizeof(P));
  for (int r = 0; r < d.R; ++r) {
    if (!z[r] || !out[r]) return PL_ERR_INVALID_ARG;
    if (((uintptr_t)z[r] & 15) || ((uintptr_t)out[r] & 15)) return PL_ERR_ALIGNMENT;
    P.y[r] = z[r];
    P.gates[r] = plan->d_ones;  // the expert layer has already applied the gates
    P.out[r] = out[r];
  }
  const unsigned long long n_tok = (unsigned long long)d.R * d.T;
  const int grid = (int)std::min<unsigned long long>(n_tok, (unsigned long long)plan->sm_count * plan->combine_per_sm);
  moe_combine_kernel<<<grid, kCombineThreads, 0, static_cast<cudaStream_t>(stream)>>>(P, d);
  if (cudaGetLastError() != cudaSuccess) return PL_ERR_CUDA;
  g_launches.fetch_add(1);
  return PL_OK;
}

pl_status_t pl_moe_plan_read_dedup(pl_moe_plan_t plan, int32_t* pos, int64_t* counts, void* stream) {
  if (!plan) return PL_ERR_INVALID_ARG;
  const MoeGeo& d = plan->gd;
  if (cudaStreamSynchronize(static_cast<cudaStream_t>(stream)) != cudaSuccess) { cudaGetLastError(); return PL_ERR_CUDA; }
  int flags[4] = {0, 0, 0, 0};
  bool ok = cudaMemcpy(flags, d.flags, 16, cudaMemcpyDeviceToHost) == cudaSuccess;
  if (ok && flags[3]) {
    flags[2] = 1;
    ok = cudaMemset(d.flags + 3, 0, 4 + 8) == cudaSuccess;
  }
  if (ok && counts) ok = cudaMemcpy(counts, d.counts, (size_t)d.R * d.R * 8, cudaMemcpyDeviceToHost) == cudaSuccess;
  if (ok && pos) {
    const size_t tk = (size_t)d.R * d.T * d.K;
    std::vector<int32_t> ridx(tk), rpos(tk);
    ok = cudaMemcpy(ridx.data(), plan->d_ridx, tk * 4, cudaMemcpyDeviceToHost) == cudaSuccess &&
         cudaMemcpy(rpos.data(), d.pos, tk * 4, cudaMemcpyDeviceToHost) == cudaSuccess;
    if (ok) {
      const size_t n_tok = (size_t)d.R * d.T;
      for (size_t i = 0; i < n_tok * d.R; ++i) pos[i] = -1;
      for (size_t t = 0; t < n_tok; ++t)
        for (int j = 0; j < d.K; ++j)
          if (ridx[t * d.K + j] >= 0) pos[t * d.R + ridx[t * d.K + j]] = rpos[t * d.K + j];
    }
  }
  if (!ok) { cudaGetLastError(); return PL_ERR_CUDA; }
  if (flags[2]) return PL_ERR_TIMEOUT;
  if (flags[1]) return PL_ERR_INVALID_ARG;
  if (flags[0]) return PL_ERR_OVERFLOW;
  return PL_OK;
}

}  // extern "C"
