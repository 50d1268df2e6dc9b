// Host orchestrator: lowers (collective, algorithm, chunk size) into a flat list of
// chunk-granular ops with wait / signal edges.  It plays the role the paper gives to its
// orchestration tier (Sec. 3.2): dependencies are derived from the input and output
// layouts (Listing 2), the composed all-reduce follows Algorithm 1 without the staging
// role, and the consume operation (copy or reduce) selects the op kind.  Everything here
// is plain host C++: no CUDA calls.
#include <algorithm>
#include <cmath>
#include <cstdio>
#include <cstring>
#include <map>
#include <numeric>

#include "pl_internal.h"

namespace pl {
namespace {

pl_ref_t ref(int rank, int buf, int dtype, uint64_t off) {
  pl_ref_t r;
  std::memset(&r, 0, sizeof(r));
  r.rank = rank;
  r.buf = buf;
  r.dtype = dtype;
  r.offset = off;
  return r;
}

struct Emitter {
  Lowered* L;
  uint32_t slice_bytes;
  int dtype = PL_U8;  // the schedule's element type
  int queues_per_rank = 1;
  // Chunks each rank runs in the phase being emitted (0 = unknown).  When known, the slice
  // count is nudged upwards so that a rank's work items divide evenly over its queues.
  uint64_t phase_chunks = 0;
  // slice_bytes == 0: the slice count is chosen per phase by a cost model, slices stay within
  // [min_slice, max_slice]
  uint32_t min_slice = 16384, max_slice = 131072;
  double op_overhead_us = 1.5, wait_overhead_us = 0.5;
  int role = 0;  // role stamped on emitted ops
  // Non-zero: COPY ops are cut into slices of exactly this many bytes (short tail), dealt
  // round-robin over the rank's queues.  Set for all-to-all on the bulk-copy datapath, where
  // every byte is read once from HBM and written once: the CTAs of a rank then sweep one
  // compact window of the source and one of the destination instead of 18 separate regions
  // (measured on B200, R = 8: 64 MiB per rank 185 -> 169 us, 256 MiB 694 -> 644 us; all-gather,
  // whose sources are re-read from L2, prefers the coarse slices of the cost model).
  uint32_t stream_slice = 0;
  // The same for the direct-fused all-reduce (a reduce whose result goes to all R outputs,
  // as many bytes written as read): slices of two ring stages, in bytes of the result
  // (measured, R = 8: 128 MiB per rank 370 -> 336 us, 256 MiB 688 -> 655 us).
  uint32_t fused_slice = 0;
  // And for the reduce ops of a large direct reduce-scatter / rooted reduce of bf16 data over 8
  // ranks, which neither wait nor signal: two ring stages of results per slice as well
  // (measured: 64 MiB per rank 98.4 -> 96.3 us, 256 MiB 370 -> 352 us = 7.06 TB/s).  Not for
  // fp32 data, other rank counts, ragged partitions or messages under 64 MiB, where the cost
  // model's coarser slices measured faster.
  uint32_t reduce_slice = 0;

  int new_flag() { return L->n_flags++; }

  // Emit one chunk-granular op.  A chunk wider than slice_bytes is cut into slices that
  // different CTAs of the executing rank run; every slice signals the chunk's flag, so the
  // flag counts finished slices and a waiter needs all of them (Sec. 3.2: the last CTA of a
  // group to finish a chunk is the one that makes it visible).
  void chunk_op(int kind, int exec_rank, int layer, pl_ref_t dst, bool bcast,
                const std::vector<pl_ref_t>& src, uint64_t count, const std::vector<int>& waits,
                int signal, int signal2 = -1) {
    int max_es = elem_size(dst.dtype);
    for (const pl_ref_t& s : src) max_es = std::max(max_es, elem_size(s.dtype));
    // elements per 16-byte vector of the schedule's element type: the kernel's unit of work,
    // which also keeps every (wider) partial operand aligned
    const uint64_t unit16 = kind == PL_OP_COPY ? 16 : 16 / elem_size(dtype);
    uint64_t wide = count * max_es;
    uint64_t n_slices = 1;
    const uint32_t fixed = slice_bytes ? 0u
                           : kind == PL_OP_COPY ? stream_slice
                           : bcast ? fused_slice
                           : (waits.empty() && signal < 0 && signal2 < 0) ? reduce_slice : 0u;
    if (fixed) {
      n_slices = std::max<uint64_t>(1, (wide + fixed - 1) / fixed);
    } else if (slice_bytes) {
      if (wide > (uint64_t)slice_bytes + slice_bytes / 2) n_slices = (wide + slice_bytes - 1) / slice_bytes;
    } else {
      // Pick the slice count that minimises the time of the phase under a simple model: a rank
      // runs `chunks` chunks of this shape on `queues_per_rank` queues; a queue spends a fixed
      // cost per op (descriptor hand-off, barrier, flag traffic: small for the bulk-copy ring,
      // which runs ahead across ops, larger for the register path) plus its bytes at the
      // per-SM share of the memory bandwidth.
      uint64_t traffic = count * elem_size(dst.dtype) * (bcast ? 8 : 1);
      for (const pl_ref_t& s : src) traffic += count * elem_size(s.dtype);
      const double chunks = (double)std::max<uint64_t>(1, phase_chunks);
      const double bytes_per_us = 40000.0;  // ~6 TB/s over 148 SMs
      const uint64_t k_lo = std::max<uint64_t>(1, (wide + max_slice - 1) / max_slice);
      const uint64_t k_hi = std::max<uint64_t>(k_lo, std::min<uint64_t>(wide / std::max<uint32_t>(16, min_slice), 8ull * queues_per_rank));
      // an op that waits on a flag cannot hide that latency behind its predecessor
      const double overhead = op_overhead_us + (waits.empty() ? 0.0 : wait_overhead_us);
      double best = 1e300;
      for (uint64_t k = k_lo; k <= k_hi; ++k) {
        const double rounds = std::ceil(chunks * (double)k / (double)queues_per_rank);
        const double cost = rounds * (overhead + (double)traffic / (double)k / bytes_per_us);
        if (cost < best * 0.97) {  // more slices only for a clear gain
          best = cost;
          n_slices = k;
        }
      }
    }
    uint64_t per = (count + n_slices - 1) / n_slices;
    uint64_t unit = (per >= 64 * unit16) ? 8 * unit16 : unit16;
    per = (per + unit - 1) / unit * unit;
    if (fixed && n_slices > 1) per = fixed / max_es;  // exact slices, short tail
    for (uint64_t b = 0; b < count; b += per) {
      HostOp op;
      op.kind = kind;
      op.exec_rank = exec_rank;
      op.layer = layer;
      op.count = std::min(per, count - b);
      op.dst = dst;
      op.dst.offset += b * elem_size(dst.dtype);
      op.bcast = bcast;
      for (pl_ref_t s : src) {
        s.offset += b * elem_size(s.dtype);
        op.src.push_back(s);
      }
      op.waits = waits;
      op.signal = signal;
      op.signal2 = signal2;
      op.role = role;
      L->ops.push_back(std::move(op));
    }
  }
};

struct Geo {
  int R, dtype, es;
  uint64_t n;            // elements per rank message
  uint64_t P;            // elements per partition
  uint64_t chunk;        // elements per chunk (clipped to P)
  uint64_t n_c;          // chunks per partition
  uint64_t clen(uint64_t c) const { return std::min(chunk, P - c * chunk); }
};

Geo make_geo(int R, int dtype, uint64_t n, uint64_t part_elems, uint64_t chunk_bytes) {
  Geo g;
  g.R = R;
  g.dtype = dtype;
  g.es = elem_size(dtype);
  g.n = n;
  g.P = part_elems;
  g.chunk = std::max<uint64_t>(1, std::min<uint64_t>(chunk_bytes / g.es, g.P));
  g.n_c = g.P ? (g.P + g.chunk - 1) / g.chunk : 0;
  return g;
}

// Cross-layer edges of a multi-layer schedule: `pub[p]` is the flag that tells that rank p's
// contribution to this layer may be read (its previous layer's output is complete), -1 when
// there is nothing to wait for; `done[r]` is the flag every op that writes rank r's output
// in this layer must signal, -1 when nobody will ask.
struct LayerEdges {
  std::vector<int> pub;
  std::vector<int> done;
};

std::vector<int> waits_on(const LayerEdges* le, const std::vector<int>& ranks) {
  std::vector<int> w;
  if (!le) return w;
  for (int p : ranks)
    if (le->pub[p] >= 0 && std::find(w.begin(), w.end(), le->pub[p]) == w.end()) w.push_back(le->pub[p]);
  return w;
}

std::vector<int> all_ranks(int R) {
  std::vector<int> v(R);
  std::iota(v.begin(), v.end(), 0);
  return v;
}

// reduce-scatter, direct: rank r reduces chunk c of partition r from all R inputs in
// ascending rank order (Listing 2: packed output => out = dst + offset, reduce waits for
// all producers; with peer-visible inputs there is nothing to wait for).
void rs_direct(Emitter& em, const Geo& g) {
  em.phase_chunks = g.n_c;
  for (uint64_t c = 0; c < g.n_c; ++c)
    for (int r = 0; r < g.R; ++r) {
      std::vector<pl_ref_t> src;
      for (int p = 0; p < g.R; ++p) src.push_back(ref(p, PL_BUF_IN, g.dtype, (r * g.P + c * g.chunk) * g.es));
      em.chunk_op(PL_OP_REDUCE, r, 0, ref(r, PL_BUF_OUT, g.dtype, c * g.chunk * g.es), false, src, g.clen(c), {}, -1);
    }
}

// all-gather, direct, as a push: rank p writes chunk c of its contribution into slot p of every
// rank's output (one load, R stores per tile; Listing 2's scattered output, out + peer*partBytes +
// offset, written by the producer).  Same result as a pull by every consumer; the contribution is
// read once instead of R times, which on one GPU takes the R-1 re-reads out of L2 and the
// load queue.  (The paper pulls because a pull over NVLink is cheaper than a push, Sec. 3.2;
// between buffers of one HBM the store count is the same either way.)
void ag_direct_push(Emitter& em, const Geo& g) {
  em.phase_chunks = g.n_c;
  for (uint64_t c = 0; c < g.n_c; ++c)
    for (int p = 0; p < g.R; ++p)
      em.chunk_op(PL_OP_COPY, p, 0, ref(p, PL_BUF_OUT, PL_U8, (p * g.P + c * g.chunk) * g.es), true,
                  {ref(p, PL_BUF_IN, PL_U8, c * g.chunk * g.es)}, g.clen(c) * g.es, {}, -1);
}

// all-to-all, direct: rank r copies partition r of every source p to slot p of its output.
void a2a_direct(Emitter& em, const Geo& g) {
  em.phase_chunks = g.n_c * g.R;
  for (uint64_t c = 0; c < g.n_c; ++c)
    for (int i = 0; i < g.R; ++i)
      for (int r = 0; r < g.R; ++r) {
        int p = (r + i) % g.R;
        uint64_t bytes = g.clen(c) * g.es;
        em.chunk_op(PL_OP_COPY, r, 0, ref(r, PL_BUF_OUT, PL_U8, (p * g.P + c * g.chunk) * g.es), false,
                    {ref(p, PL_BUF_IN, PL_U8, (r * g.P + c * g.chunk) * g.es)}, bytes, {}, -1);
      }
}

// all-to-all-v: counts[p][r] elements from p to r; sender offsets are prefix sums over
// destinations, receiver offsets prefix sums over sources (transposedV layout).
void a2av_direct(Emitter& em, int R, int dtype, const uint64_t* counts, uint64_t chunk_bytes) {
  const int es = elem_size(dtype);
  std::vector<uint64_t> soff(R * R), roff(R * R);
  for (int p = 0; p < R; ++p) {
    uint64_t a = 0;
    for (int r = 0; r < R; ++r) { soff[p * R + r] = a; a += counts[p * R + r]; }
  }
  for (int r = 0; r < R; ++r) {
    uint64_t a = 0;
    for (int p = 0; p < R; ++p) { roff[p * R + r] = a; a += counts[p * R + r]; }
  }
  uint64_t max_seg = 0;
  for (int i = 0; i < R * R; ++i) max_seg = std::max(max_seg, counts[i] * es);
  uint64_t chunk = std::max<uint64_t>(16, chunk_bytes);
  uint64_t busiest = 1;  // chunk ops of the rank that receives the most
  for (int r = 0; r < R; ++r) {
    uint64_t c = 0;
    for (int p = 0; p < R; ++p) c += (counts[p * R + r] * es + chunk - 1) / chunk;
    busiest = std::max(busiest, c);
  }
  em.phase_chunks = busiest;
  for (uint64_t b = 0; b < max_seg; b += chunk)
    for (int i = 0; i < R; ++i)
      for (int r = 0; r < R; ++r) {
        int p = (r + i) % R;
        uint64_t seg = counts[p * R + r] * es;
        if (b >= seg) continue;
        uint64_t bytes = std::min(chunk, seg - b);
        em.chunk_op(PL_OP_COPY, r, 0, ref(r, PL_BUF_OUT, PL_U8, roff[p * R + r] * es + b), false,
                    {ref(p, PL_BUF_IN, PL_U8, soff[p * R + r] * es + b)}, bytes, {}, -1);
      }
}

// reduce-scatter-v / all-gather-v: the fixed-size rules with run-time partition sizes n[k]
// (offsets are prefix sums, Sec. 3.1 "V variants").
void rsv_direct(Emitter& em, int R, int dtype, const uint64_t* n, uint64_t chunk_bytes) {
  const int es = elem_size(dtype);
  const uint64_t chunk = std::max<uint64_t>(16 / es, chunk_bytes / es);
  uint64_t max_n = 0;
  std::vector<uint64_t> off(R, 0);
  for (int k = 0; k < R; ++k) { max_n = std::max(max_n, n[k]); if (k) off[k] = off[k - 1] + n[k - 1]; }
  em.phase_chunks = std::max<uint64_t>(1, (max_n + chunk - 1) / chunk);  // chunk ops of the busiest rank
  for (uint64_t b = 0; b < max_n; b += chunk)
    for (int k = 0; k < R; ++k) {
      if (b >= n[k]) continue;
      std::vector<pl_ref_t> src;
      for (int p = 0; p < R; ++p) src.push_back(ref(p, PL_BUF_IN, dtype, (off[k] + b) * es));
      em.chunk_op(PL_OP_REDUCE, k, 0, ref(k, PL_BUF_OUT, dtype, b * es), false, src, std::min(chunk, n[k] - b), {}, -1);
    }
}

void agv_direct(Emitter& em, int R, int dtype, const uint64_t* n, uint64_t chunk_bytes) {
  const int es = elem_size(dtype);
  const uint64_t chunk = std::max<uint64_t>(16, chunk_bytes);
  uint64_t max_b = 0;
  std::vector<uint64_t> off(R, 0);
  for (int p = 0; p < R; ++p) {
    max_b = std::max(max_b, n[p] * es);
    if (p) off[p] = off[p - 1] + n[p - 1] * es;
  }
  // chunk ops per rank: its own contribution
  em.phase_chunks = std::max<uint64_t>(1, (max_b + chunk - 1) / chunk);
  // rank p writes its contribution into every output (see ag_direct_push)
  for (uint64_t b = 0; b < max_b; b += chunk)
    for (int p = 0; p < R; ++p) {
      if (b >= n[p] * es) continue;
      em.chunk_op(PL_OP_COPY, p, 0, ref(p, PL_BUF_OUT, PL_U8, off[p] + b), true, {ref(p, PL_BUF_IN, PL_U8, b)},
                  std::min(chunk, n[p] * es - b), {}, -1);
    }
}

// ---- rooted collectives (Appendix B of the paper: layouts plus a Root role) ----------------
// scatter: only the root produces; rank r copies partition r of the root's input.
void scatter_direct(Emitter& em, const Geo& g, int root) {
  em.phase_chunks = g.n_c;
  for (uint64_t c = 0; c < g.n_c; ++c)
    for (int r = 0; r < g.R; ++r)
      em.chunk_op(PL_OP_COPY, r, 0, ref(r, PL_BUF_OUT, PL_U8, c * g.chunk * g.es), false,
                  {ref(root, PL_BUF_IN, PL_U8, (r * g.P + c * g.chunk) * g.es)}, g.clen(c) * g.es, {}, -1);
}

// gather: only the root consumes.  Rank p writes its packed contribution into slot p of the
// root's output (a push): the copies then run on every rank's queues.  Left to the root as
// pulls they would all sit on the root's queues, one eighth of the CTAs at R = 8.
void gather_direct(Emitter& em, const Geo& g, int root) {
  em.phase_chunks = g.n_c;
  for (uint64_t c = 0; c < g.n_c; ++c)
    for (int p = 0; p < g.R; ++p)
      em.chunk_op(PL_OP_COPY, p, 0, ref(root, PL_BUF_OUT, PL_U8, (p * g.P + c * g.chunk) * g.es), false,
                  {ref(p, PL_BUF_IN, PL_U8, c * g.chunk * g.es)}, g.clen(c) * g.es, {}, -1);
}

// broadcast = compose<scatter, all-gather> with both copies folded into one op: rank k takes
// chunk c of partition k from the root's input (the scatter) and writes it into every rank's
// output (the all-gather, as a push).  One phase, no flags, every rank's queues share the work;
// the root's buffer is read once.
void broadcast_composed(Emitter& em, const Geo& g, int root) {
  em.phase_chunks = g.n_c;
  for (uint64_t c = 0; c < g.n_c; ++c)
    for (int k = 0; k < g.R; ++k) {
      const uint64_t off = (k * g.P + c * g.chunk) * g.es;
      em.chunk_op(PL_OP_COPY, k, 0, ref(k, PL_BUF_OUT, PL_U8, off), true, {ref(root, PL_BUF_IN, PL_U8, off)},
                  g.clen(c) * g.es, {}, -1);
    }
}

// reduce = compose<reduce-scatter, gather>: rank k reduces chunk c of partition k (ascending
// rank order) and, the gather being a push, writes the result straight into partition k of
// the root's output: one pass, no intermediate buffer, no flags.
void reduce_composed(Emitter& em, const Geo& g, int root) {
  em.phase_chunks = g.n_c;
  for (uint64_t c = 0; c < g.n_c; ++c)
    for (int k = 0; k < g.R; ++k) {
      std::vector<pl_ref_t> src;
      const uint64_t off = (k * g.P + c * g.chunk) * g.es;
      for (int p = 0; p < g.R; ++p) src.push_back(ref(p, PL_BUF_IN, g.dtype, off));
      em.chunk_op(PL_OP_REDUCE, k, 0, ref(root, PL_BUF_OUT, g.dtype, off), false, src, g.clen(c), {}, -1);
    }
}

// all-reduce, one-shot: every rank reduces the whole message from all R inputs.
void ar_oneshot(Emitter& em, const Geo& g, int layer, uint64_t in_off, uint64_t out_off, const LayerEdges* le) {
  // g.P == g.n here: the "partition" is the whole message, chunked.
  em.phase_chunks = g.n_c;
  for (uint64_t c = 0; c < g.n_c; ++c)
    for (int r = 0; r < g.R; ++r) {
      std::vector<pl_ref_t> src;
      for (int p = 0; p < g.R; ++p) src.push_back(ref(p, PL_BUF_IN, g.dtype, in_off + c * g.chunk * g.es));
      em.chunk_op(PL_OP_REDUCE, r, layer, ref(r, PL_BUF_OUT, g.dtype, out_off + c * g.chunk * g.es), false, src,
                  g.clen(c), waits_on(le, all_ranks(g.R)), le ? le->done[r] : -1);
    }
}

// Layered one-shot all-reduce for the packet datapath (Sec. 3.2, "Specializing for latency").
// Rank r is a group of G CTAs; CTA (r, j) reduces slice j of every layer's message from all R
// contributions.  The op list states the data movement and the ordering rules, with logical
// flags: done[r][l] is signalled by the G ops of rank r in layer l and every op of layer l+1
// waits for done[p][l] of all p (rank p's contribution to layer l+1 counts as published once
// p's layer-l output is complete).  On the device no flag word exists: the G CTAs of a rank
// join with a cluster barrier, then copy their slice of the next layer's input into 16-byte
// packets (8 B payload + 8 B layer tag), and consumers poll the packets themselves.
void ar_oneshot_packets(Emitter& em, const Geo& g, int n_layers, int G) {
  const int R = g.R;
  const uint64_t msg = g.n * g.es, per = g.n / (uint64_t)G;
  std::vector<int> prev, cur;
  for (int l = 0; l < n_layers; ++l) {
    cur.assign(R, -1);
    if (l + 1 < n_layers)
      for (int r = 0; r < R; ++r) cur[r] = em.new_flag();
    for (int r = 0; r < R; ++r)
      for (int j = 0; j < G; ++j) {
        HostOp op;
        op.kind = PL_OP_REDUCE;
        op.exec_rank = r;
        op.layer = l;
        op.count = per;
        const uint64_t off = (uint64_t)l * msg + (uint64_t)j * per * g.es;
        op.dst = ref(r, PL_BUF_OUT, g.dtype, off);
        for (int p = 0; p < R; ++p) op.src.push_back(ref(p, PL_BUF_IN, g.dtype, off));
        if (l > 0) op.waits = prev;
        op.signal = cur[r];
        op.queue = j * R + r;
        em.L->ops.push_back(std::move(op));
      }
    prev = cur;
  }
  em.L->queues_preassigned = true;
  // two packet buffers per rank, alternated by layer parity, each the message as packets (2x)
  for (int r = 0; r < R; ++r) em.L->scratch_per_rank[r] = 4 * msg;
}

// all-reduce, direct fused: the reducer of partition k writes each result into all R outputs.
void ar_fused(Emitter& em, const Geo& g, int layer, uint64_t in_off, uint64_t out_off, const LayerEdges* le) {
  em.phase_chunks = g.n_c;
  for (uint64_t c = 0; c < g.n_c; ++c)
    for (int k = 0; k < g.R; ++k) {
      std::vector<pl_ref_t> src;
      uint64_t off = (k * g.P + c * g.chunk) * g.es;
      for (int p = 0; p < g.R; ++p) src.push_back(ref(p, PL_BUF_IN, g.dtype, in_off + off));
      // every output is complete only when every reducer is: one shared flag per layer
      em.chunk_op(PL_OP_REDUCE, k, layer, ref(k, PL_BUF_OUT, g.dtype, out_off + off), true, src, g.clen(c),
                  waits_on(le, all_ranks(g.R)), le ? le->done[0] : -1);
    }
}

// all-reduce, direct two-shot = compose<reduce-scatter, all-gather> in one launch
// (Algorithm 1 without the staging role): rank k reduces chunk c of partition k into its own
// output and publishes reduced(k,c) to all ranks; every other rank then copies that chunk.
void ar_direct(Emitter& em, const Geo& g, int layer, uint64_t in_off, uint64_t out_off, const LayerEdges* le) {
  std::vector<int> reduced(g.R * g.n_c);
  em.phase_chunks = g.n_c;
  for (uint64_t c = 0; c < g.n_c; ++c)
    for (int k = 0; k < g.R; ++k) {
      int f = reduced[k * g.n_c + c] = em.new_flag();
      std::vector<pl_ref_t> src;
      uint64_t off = (k * g.P + c * g.chunk) * g.es;
      for (int p = 0; p < g.R; ++p) src.push_back(ref(p, PL_BUF_IN, g.dtype, in_off + off));
      em.chunk_op(PL_OP_REDUCE, k, layer, ref(k, PL_BUF_OUT, g.dtype, out_off + off), false, src, g.clen(c),
                  waits_on(le, all_ranks(g.R)), f, le ? le->done[k] : -1);
    }
  em.phase_chunks = g.n_c * (g.R - 1);
  for (uint64_t c = 0; c < g.n_c; ++c)
    for (int i = 1; i < g.R; ++i)
      for (int r = 0; r < g.R; ++r) {
        int k = (r + i) % g.R;
        uint64_t off = (k * g.P + c * g.chunk) * g.es;
        em.chunk_op(PL_OP_COPY, r, layer, ref(r, PL_BUF_OUT, PL_U8, out_off + off), false,
                    {ref(k, PL_BUF_OUT, PL_U8, out_off + off)}, g.clen(c) * g.es, {reduced[k * g.n_c + c]},
                    le ? le->done[r] : -1);
      }
}

// Ring reduce-scatter.  Partition k's chain starts with rank k+1's own input and visits
// k+2, ..., k (mod R).  At step s in [0, R-2] rank r handles k = (r - s - 2) mod R:
//   part_r[k] = part_{r-1}[k] + in_r[k]      (step 0 reads in_{r-1}[k] directly)
// and the last step writes rank r's result.  Partials are kept in the partial dtype
// (fp32 for bf16 data) in per-step scratch slots.  `final_to_out_partition`: write the last
// hop to out_r + r*P (all-reduce) instead of out_r + 0 (reduce-scatter).  Returns the flag
// of (r, last step, c) in final_flags when asked.
void rs_ring(Emitter& em, const Geo& g, bool final_to_out_partition, std::vector<int>* final_flags) {
  const int R = g.R, pd = partial_dtype(g.dtype), ps = elem_size(pd);
  std::vector<int> prev(R * g.n_c, -1), cur(R * g.n_c, -1);
  em.phase_chunks = g.n_c;
  for (int s = 0; s <= R - 2; ++s) {
    const bool last = (s == R - 2);
    for (uint64_t c = 0; c < g.n_c; ++c)
      for (int r = 0; r < R; ++r) {
        const int k = ((r - s - 2) % R + R) % R, q = (r - 1 + R) % R;
        const uint64_t in_off = (k * g.P + c * g.chunk) * g.es;
        pl_ref_t a = (s == 0) ? ref(q, PL_BUF_IN, g.dtype, in_off)
                              : ref(q, PL_BUF_SCRATCH, pd, ((s - 1) * g.P + c * g.chunk) * ps);
        pl_ref_t b = ref(r, PL_BUF_IN, g.dtype, in_off);
        pl_ref_t d = last ? ref(r, PL_BUF_OUT, g.dtype, ((final_to_out_partition ? r * g.P : 0) + c * g.chunk) * g.es)
                          : ref(r, PL_BUF_SCRATCH, pd, (s * g.P + c * g.chunk) * ps);
        std::vector<int> w;
        if (s > 0) w.push_back(prev[q * g.n_c + c]);
        int f = -1;
        if (!last || final_flags) f = em.new_flag();
        cur[r * g.n_c + c] = f;
        em.chunk_op(PL_OP_COPY_REDUCE, r, 0, d, false, {a, b}, g.clen(c), w, f);
      }
    prev = cur;
  }
  if (final_flags) *final_flags = prev;
  if (R > 2)
    for (int r = 0; r < R; ++r) em.L->scratch_per_rank[r] = (uint64_t)(R - 2) * g.P * ps;
}

// Ring all-gather.  Rank r first places its own contribution, then at step s in [0, R-2]
// copies partition (r - s - 1) mod R from rank r-1 (from r-1's input at step 0, from its
// output afterwards).  `own_from_out`: the own partition already sits in out_r (all-reduce);
// own_flags then carries the flags that say so.
void ag_ring(Emitter& em, const Geo& g, bool own_from_out, const std::vector<int>* own_flags) {
  const int R = g.R;
  std::vector<int> prev(R * g.n_c, -1), cur(R * g.n_c, -1);
  em.phase_chunks = g.n_c;
  if (!own_from_out)
    for (uint64_t c = 0; c < g.n_c; ++c)
      for (int r = 0; r < R; ++r)
        em.chunk_op(PL_OP_COPY, r, 0, ref(r, PL_BUF_OUT, PL_U8, (r * g.P + c * g.chunk) * g.es), false,
                    {ref(r, PL_BUF_IN, PL_U8, c * g.chunk * g.es)}, g.clen(c) * g.es, {}, -1);
  for (int s = 0; s <= R - 2; ++s) {
    for (uint64_t c = 0; c < g.n_c; ++c)
      for (int r = 0; r < R; ++r) {
        const int k = ((r - s - 1) % R + R) % R, q = (r - 1 + R) % R;
        const uint64_t off = (k * g.P + c * g.chunk) * g.es;
        pl_ref_t src = (s == 0 && !own_from_out) ? ref(q, PL_BUF_IN, PL_U8, c * g.chunk * g.es)
                                                 : ref(q, PL_BUF_OUT, PL_U8, off);
        std::vector<int> w;
        if (s == 0) {
          if (own_from_out) w.push_back((*own_flags)[q * g.n_c + c]);
        } else {
          w.push_back(prev[q * g.n_c + c]);
        }
        int f = (s < R - 2) ? em.new_flag() : -1;
        cur[r * g.n_c + c] = f;
        em.chunk_op(PL_OP_COPY, r, 0, ref(r, PL_BUF_OUT, PL_U8, off), false, {src}, g.clen(c) * g.es, w, f);
      }
    prev = cur;
  }
}

// Binomial-tree all-reduce, chunk-pipelined.  Reduce: at level l every rank r that is a
// multiple of 2^(l+1) adds the running sum of rank r + 2^l (skipped when that rank does not
// exist) to its own; running sums live in fp32 scratch (one slot per level, never
// overwritten); the root's last addition writes the output.  Broadcast: the same tree in
// reverse, child r + 2^l copies the finished chunk from r's output.
void ar_tree(Emitter& em, const Geo& g) {
  // Binomial reduce to a root, then binomial broadcast from it, pipelined over chunks of the
  // whole message (g.P == g.n).  The tree is built over virtual ranks v = (r - root) mod R and
  // the root rotates with the chunk index, so that every rank's queues carry the same load: a
  // fixed root would leave its CTAs with log2(R) full passes over the message while the leaves'
  // idle.  A single chunk gives the textbook tree rooted at rank 0.
  const int R = g.R, pd = partial_dtype(g.dtype), ps = elem_size(pd);
  int levels = 0;
  while ((1 << levels) < R) ++levels;
  // chunk-level ops a rank runs in all: 2(R-1) per chunk, shared evenly by the rotation
  em.phase_chunks = std::max<uint64_t>(1, g.n_c * 2 * (uint64_t)(R - 1) / (uint64_t)R);
  // Scratch slot l of a rank holds what it produced at level l (the root's last level writes
  // the output instead).
  std::vector<int> slots(R, 0);
  // Ops are stored by wavefront (chunk index + D * stage): a queue then meets the stages of
  // successive chunks in the order in which their inputs become ready.  The skew D leaves a
  // stage's inputs D chunks of head start; with D = 1 queue heads regularly sat waiting on a
  // flag with runnable ops behind them (measured on B200, 64 MiB per rank, R = 8: 838 us at
  // D = 1, 472 us at D = 8, against 470 us for the ring).
  const uint64_t D = (uint64_t)R;
  std::vector<std::vector<HostOp>> wave(g.n_c + 2 * (size_t)levels * D);
  const size_t base_ops = em.L->ops.size();
  auto stash = [&](uint64_t key) {
    auto& ops = em.L->ops;
    for (size_t i = base_ops; i < ops.size(); ++i) wave[key].push_back(std::move(ops[i]));
    ops.resize(base_ops);
  };
  for (uint64_t c = 0; c < g.n_c; ++c) {
    const int root = (int)(c % (uint64_t)R);
    auto phys = [&](int v) { return (v + root) % R; };
    std::vector<pl_ref_t> acc(R);     // by virtual rank: where its running sum of chunk c lives
    std::vector<int> acc_flag(R, -1);
    std::vector<int> has(R, -1);      // by virtual rank: "out chunk c is final"
    for (int v = 0; v < R; ++v) acc[v] = ref(phys(v), PL_BUF_IN, g.dtype, c * g.chunk * g.es);
    for (int l = 0; l < levels; ++l) {
      for (int v = 0; v < R; v += (1 << (l + 1))) {
        const int q = v + (1 << l);
        if (q >= R) continue;
        const bool to_out = (v == 0 && l == levels - 1);
        const int r = phys(v);
        pl_ref_t d = to_out ? ref(r, PL_BUF_OUT, g.dtype, c * g.chunk * g.es)
                            : ref(r, PL_BUF_SCRATCH, pd, ((uint64_t)l * g.n + c * g.chunk) * ps);
        if (!to_out) slots[r] = std::max(slots[r], l + 1);
        std::vector<int> w;
        if (acc_flag[v] >= 0) w.push_back(acc_flag[v]);
        if (acc_flag[q] >= 0) w.push_back(acc_flag[q]);
        const int f = em.new_flag();
        em.chunk_op(PL_OP_COPY_REDUCE, r, 0, d, false, {acc[v], acc[q]}, g.clen(c), w, f);
        acc_flag[v] = f;
        acc[v] = d;
        if (to_out) has[0] = f;
      }
      stash(c + l * D);
    }
    for (int l = levels - 1; l >= 0; --l) {
      for (int v = 0; v < R; v += (1 << (l + 1))) {
        const int q = v + (1 << l);
        if (q >= R) continue;
        const int f = em.new_flag();
        em.chunk_op(PL_OP_COPY, phys(q), 0, ref(phys(q), PL_BUF_OUT, PL_U8, c * g.chunk * g.es), false,
                    {ref(phys(v), PL_BUF_OUT, PL_U8, c * g.chunk * g.es)}, g.clen(c) * g.es, {has[v]}, f);
        has[q] = f;
      }
      stash(c + (levels + (levels - 1 - l)) * D);
    }
  }
  for (auto& w : wave)
    for (HostOp& op : w) em.L->ops.push_back(std::move(op));
  for (int r = 0; r < R; ++r) em.L->scratch_per_rank[r] = (uint64_t)slots[r] * g.n * ps;
}

// ---- staged variants: ordinary application buffers (Sec. 3.2 protocol, Algorithm 1) --------
// Peers never touch in/out: every rank copies its contribution chunk by chunk into its own
// staging memory (stage role) and publishes it; consumers pull from staging only.  Staging has
// `ns` chunk slots per partition; chunk c lives in slot c % ns and a stage op for chunk c waits
// until chunk c - ns has been consumed (cyclic staging, Sec. 4.1).  Roles get their own CTA
// groups so that staging runs ahead of reduction and gathering.
struct Staging {
  uint64_t ns;      // chunk slots per partition
  uint64_t chunkB;  // bytes per chunk slot
};

Staging staging_geo(const Geo& g, uint64_t capacity, uint64_t partitions) {
  Staging s;
  s.chunkB = g.chunk * g.es;
  if (capacity == 0) capacity = 256ull << 20;
  s.ns = std::max<uint64_t>(1, std::min<uint64_t>(g.n_c, capacity / std::max<uint64_t>(1, partitions * s.chunkB)));
  return s;
}

void set_roles(Emitter& em, int R, const double (&cost)[4]) {
  // split a rank's queues between the roles in proportion to the bytes each role moves
  const int Q = em.queues_per_rank;
  int n_roles = 0;
  double total = 0;
  for (int i = 1; i < 4; ++i)
    if (cost[i] > 0) { ++n_roles; total += cost[i]; }
  if (Q < n_roles) return;  // too few queues: every op may run anywhere
  int left = Q;
  for (int i = 1; i < 4; ++i)
    if (cost[i] > 0) {
      em.L->role_queues[i] = std::max(1, (int)(Q * cost[i] / total));
      left -= em.L->role_queues[i];
    }
  for (int i = 1; left != 0; i = i % 3 + 1)  // hand out / take back the rounding remainder
    if (cost[i] > 0 && (left > 0 || em.L->role_queues[i] > 1)) {
      em.L->role_queues[i] += left > 0 ? 1 : -1;
      left += left > 0 ? -1 : 1;
    }
  (void)R;
}

void begin_role(Emitter& em, int role, uint64_t phase_chunks) {
  em.role = em.L->role_queues[role] ? role : 0;
  em.phase_chunks = phase_chunks;
}

void ar_direct_staged(Emitter& em, const Geo& g, uint64_t capacity) {
  const int R = g.R;
  const Staging st = staging_geo(g, capacity, R);
  // shares measured on B200 (R=8, 64 MiB): stage 8, reduce 4, gather 6 of 18 queues; the gather
  // role reads what the reducers just wrote (L2) and is cheaper than its byte count suggests
  const double cost[4] = {0, 2.0, 1.0, 1.5};
  set_roles(em, R, cost);
  const int q_all = em.queues_per_rank;
  auto S_off = [&](int k, uint64_t c) { return ((uint64_t)k * st.ns + c % st.ns) * st.chunkB; };
  auto Y_off = [&](uint64_t c) { return ((uint64_t)R * st.ns + c % st.ns) * st.chunkB; };
  std::vector<int> staged(R * g.n_c), reduced(R * g.n_c), consumed(R * g.n_c);
  for (size_t i = 0; i < staged.size(); ++i) { staged[i] = em.new_flag(); reduced[i] = em.new_flag(); consumed[i] = em.new_flag(); }
  for (uint64_t c = 0; c < g.n_c; ++c) {
    begin_role(em, 1, (uint64_t)R);
    if (em.role) em.queues_per_rank = em.L->role_queues[1];
    for (int k = 0; k < R; ++k)
      for (int r = 0; r < R; ++r) {
        std::vector<int> w;
        if (c >= st.ns) w.push_back(reduced[k * g.n_c + c - st.ns]);  // slot still holds live data
        em.chunk_op(PL_OP_COPY, r, 0, ref(r, PL_BUF_SCRATCH, PL_U8, S_off(k, c)), false,
                    {ref(r, PL_BUF_IN, PL_U8, (k * g.P + c * g.chunk) * g.es)}, g.clen(c) * g.es, w, staged[k * g.n_c + c]);
      }
    begin_role(em, 2, 1);
    if (em.role) em.queues_per_rank = em.L->role_queues[2];
    for (int k = 0; k < R; ++k) {
      std::vector<pl_ref_t> src;
      for (int p = 0; p < R; ++p) src.push_back(ref(p, PL_BUF_SCRATCH, g.dtype, S_off(k, c)));
      std::vector<int> w{staged[k * g.n_c + c]};
      if (c >= st.ns) w.push_back(consumed[k * g.n_c + c - st.ns]);
      em.chunk_op(PL_OP_REDUCE, k, 0, ref(k, PL_BUF_SCRATCH, g.dtype, Y_off(c)), false, src, g.clen(c), w, reduced[k * g.n_c + c]);
    }
    begin_role(em, 3, (uint64_t)R);
    if (em.role) em.queues_per_rank = em.L->role_queues[3];
    for (int i = 0; i < R; ++i)
      for (int r = 0; r < R; ++r) {
        const int k = (r + i) % R;
        em.chunk_op(PL_OP_COPY, r, 0, ref(r, PL_BUF_OUT, PL_U8, (k * g.P + c * g.chunk) * g.es), false,
                    {ref(k, PL_BUF_SCRATCH, PL_U8, Y_off(c))}, g.clen(c) * g.es, {reduced[k * g.n_c + c]},
                    consumed[k * g.n_c + c]);
      }
    em.queues_per_rank = q_all;
  }
  for (int r = 0; r < R; ++r) em.L->scratch_per_rank[r] = ((uint64_t)R * st.ns + st.ns) * st.chunkB;
}

void rs_direct_staged(Emitter& em, const Geo& g, uint64_t capacity) {
  const int R = g.R;
  const Staging st = staging_geo(g, capacity, R);
  const double cost[4] = {0, 1.25, 1.0, 0};  // measured: 10 staging and 8 reducing queues of 18
  set_roles(em, R, cost);
  const int q_all = em.queues_per_rank;
  auto S_off = [&](int k, uint64_t c) { return ((uint64_t)k * st.ns + c % st.ns) * st.chunkB; };
  std::vector<int> staged(R * g.n_c), reduced(R * g.n_c);
  for (size_t i = 0; i < staged.size(); ++i) { staged[i] = em.new_flag(); reduced[i] = em.new_flag(); }
  for (uint64_t c = 0; c < g.n_c; ++c) {
    begin_role(em, 1, (uint64_t)R);
    if (em.role) em.queues_per_rank = em.L->role_queues[1];
    for (int k = 0; k < R; ++k)
      for (int r = 0; r < R; ++r) {
        std::vector<int> w;
        if (c >= st.ns) w.push_back(reduced[k * g.n_c + c - st.ns]);
        em.chunk_op(PL_OP_COPY, r, 0, ref(r, PL_BUF_SCRATCH, PL_U8, S_off(k, c)), false,
                    {ref(r, PL_BUF_IN, PL_U8, (k * g.P + c * g.chunk) * g.es)}, g.clen(c) * g.es, w, staged[k * g.n_c + c]);
      }
    begin_role(em, 2, 1);
    if (em.role) em.queues_per_rank = em.L->role_queues[2];
    for (int k = 0; k < R; ++k) {
      std::vector<pl_ref_t> src;
      for (int p = 0; p < R; ++p) src.push_back(ref(p, PL_BUF_SCRATCH, g.dtype, S_off(k, c)));
      em.chunk_op(PL_OP_REDUCE, k, 0, ref(k, PL_BUF_OUT, g.dtype, c * g.chunk * g.es), false, src, g.clen(c),
                  {staged[k * g.n_c + c]}, reduced[k * g.n_c + c]);
    }
    em.queues_per_rank = q_all;
  }
  for (int r = 0; r < R; ++r) em.L->scratch_per_rank[r] = (uint64_t)R * st.ns * st.chunkB;
}

void ag_direct_staged(Emitter& em, const Geo& g, uint64_t capacity) {
  const int R = g.R;
  const Staging st = staging_geo(g, capacity, 1);
  const double cost[4] = {0, 2.0, 0, 2.0 * R};
  set_roles(em, R, cost);
  const int q_all = em.queues_per_rank;
  std::vector<int> staged(R * g.n_c), consumed(R * g.n_c);
  for (size_t i = 0; i < staged.size(); ++i) { staged[i] = em.new_flag(); consumed[i] = em.new_flag(); }
  for (uint64_t c = 0; c < g.n_c; ++c) {
    begin_role(em, 1, 1);
    if (em.role) em.queues_per_rank = em.L->role_queues[1];
    for (int r = 0; r < R; ++r) {
      std::vector<int> w;
      if (c >= st.ns) w.push_back(consumed[r * g.n_c + c - st.ns]);
      em.chunk_op(PL_OP_COPY, r, 0, ref(r, PL_BUF_SCRATCH, PL_U8, (c % st.ns) * st.chunkB), false,
                  {ref(r, PL_BUF_IN, PL_U8, c * g.chunk * g.es)}, g.clen(c) * g.es, w, staged[r * g.n_c + c]);
    }
    begin_role(em, 3, (uint64_t)R);
    if (em.role) em.queues_per_rank = em.L->role_queues[3];
    for (int i = 0; i < R; ++i)
      for (int r = 0; r < R; ++r) {
        const int p = (r + i) % R;
        em.chunk_op(PL_OP_COPY, r, 0, ref(r, PL_BUF_OUT, PL_U8, (p * g.P + c * g.chunk) * g.es), false,
                    {ref(p, PL_BUF_SCRATCH, PL_U8, (c % st.ns) * st.chunkB)}, g.clen(c) * g.es, {staged[p * g.n_c + c]},
                    consumed[p * g.n_c + c]);
      }
    em.queues_per_rank = q_all;
  }
  for (int r = 0; r < R; ++r) em.L->scratch_per_rank[r] = st.ns * st.chunkB;
}

void a2a_direct_staged(Emitter& em, const Geo& g, uint64_t capacity) {
  const int R = g.R;
  const Staging st = staging_geo(g, capacity, R);
  const double cost[4] = {0, 4.0, 0, 5.0};  // measured: 8 staging and 10 consuming queues of 18
  set_roles(em, R, cost);
  const int q_all = em.queues_per_rank;
  auto S_off = [&](int k, uint64_t c) { return ((uint64_t)k * st.ns + c % st.ns) * st.chunkB; };
  std::vector<int> staged((size_t)R * R * g.n_c), consumed((size_t)R * R * g.n_c);
  for (size_t i = 0; i < staged.size(); ++i) { staged[i] = em.new_flag(); consumed[i] = em.new_flag(); }
  auto fi = [&](int r, int k, uint64_t c) { return ((size_t)r * R + k) * g.n_c + c; };
  for (uint64_t c = 0; c < g.n_c; ++c) {
    begin_role(em, 1, (uint64_t)R);
    if (em.role) em.queues_per_rank = em.L->role_queues[1];
    for (int k = 0; k < R; ++k)
      for (int r = 0; r < R; ++r) {
        std::vector<int> w;
        if (c >= st.ns) w.push_back(consumed[fi(r, k, c - st.ns)]);
        em.chunk_op(PL_OP_COPY, r, 0, ref(r, PL_BUF_SCRATCH, PL_U8, S_off(k, c)), false,
                    {ref(r, PL_BUF_IN, PL_U8, (k * g.P + c * g.chunk) * g.es)}, g.clen(c) * g.es, w, staged[fi(r, k, c)]);
      }
    begin_role(em, 3, (uint64_t)R);
    if (em.role) em.queues_per_rank = em.L->role_queues[3];
    for (int i = 0; i < R; ++i)
      for (int k = 0; k < R; ++k) {
        const int r = (k + i) % R;  // source rank
        em.chunk_op(PL_OP_COPY, k, 0, ref(k, PL_BUF_OUT, PL_U8, (r * g.P + c * g.chunk) * g.es), false,
                    {ref(r, PL_BUF_SCRATCH, PL_U8, S_off(k, c))}, g.clen(c) * g.es, {staged[fi(r, k, c)]},
                    consumed[fi(r, k, c)]);
      }
    em.queues_per_rank = q_all;
  }
  for (int r = 0; r < R; ++r) em.L->scratch_per_rank[r] = (uint64_t)R * st.ns * st.chunkB;
}

}  // namespace

// Default knobs for sm_100a ("codesign policy", Sec. 3.2-3.3).  Called twice by the build:
// first with max_resident_ctas == 0 to settle the datapath and its shared-memory ring (which
// decide how many CTAs fit on an SM), then with the resulting capacity to settle the grid.
Policy default_policy(const BuildRequest& rq, int max_resident_ctas) {
  Policy p = rq.pol;
  const int es = elem_size(rq.dtype);
  uint64_t msg = rq.count_per_rank * es;
  if (rq.counts_v) {
    msg = 0;
    const int entries = rq.coll == PL_ALLTOALLV ? rq.R * rq.R : rq.R;
    for (int i = 0; i < entries; ++i) msg += rq.counts_v[i] * es;
    if (rq.coll == PL_ALLTOALLV) msg /= rq.R;
  }
  if (rq.coll == PL_ALLGATHER) msg *= rq.R;
  // bytes of all ranks' inputs and outputs: decides whether the working set lives in L2
  uint64_t footprint = 2 * (uint64_t)rq.R * msg;
  if (rq.coll == PL_REDUCE_SCATTER || rq.coll == PL_ALLGATHER || rq.coll == PL_REDUCE_SCATTERV || rq.coll == PL_ALLGATHERV)
    footprint = (uint64_t)(rq.R + 1) * msg;
  if (rq.coll == PL_ALLTOALLV) footprint = 2 * (uint64_t)rq.R * msg;
  // Register path while the working set is L2 sized (and for layered latency schedules);
  // bulk-copy ring once it has to stream from HBM.  Measured crossovers on B200 at R=8
  // (128-call CUDA graphs): reduce-scatter, all-gather, all-to-all, scatter, gather, broadcast
  // between 72 and 144 MiB of inputs + outputs (the L2 holds 126 MB); all-reduce between 128
  // and 256 MiB (its outputs are written once and never re-read).
  const uint64_t knee = rq.coll == PL_ALLREDUCE ? (256ull << 20) : (128ull << 20);
  const bool stream = footprint >= knee && rq.n_layers == 0;
  if (p.datapath == PL_DP_AUTO) p.datapath = stream ? PL_DP_TMA : PL_DP_LDST;
  if (p.threads <= 0) p.threads = 512;
  if (p.stages <= 0) p.stages = 4;
  // 48 KiB slots hold a full stage of 384 units of 8 sources; with a second operand per rank its
  // tile rides in the slot as a ninth one, and 54 KiB keep the stage at 384 units (the general
  // consumer path costs about a microsecond per stage whatever its size: reduce-scatter with
  // residual 119 -> 111 us at 8 x 64 MiB; not the ring, whose stages hold partial sums and lose 2 %)
  if (p.stage_bytes == 0) p.stage_bytes = ((rq.hook & PL_HOOK_RESIDUAL) && rq.algo != PL_ALGO_RING) ? 55296 : 49152;
  // Latency regime (at most 1 MiB per rank, and every layered schedule): slices down to 2 KiB,
  // one work item per queue, as many queues as there are items.  Measured on B200 with 80
  // layers in one launch: 16 KiB one-shot is fastest with 8 queues per rank of 2 KiB each.
  const bool latency = msg <= (1u << 20) || rq.n_layers > 0;
  p.min_slice = latency ? 2048 : 16384;
  p.max_slice = latency ? 32768 : (p.datapath == PL_DP_TMA ? 262144 : 131072);
  if (max_resident_ctas <= 0) return p;
  if (p.n_ctas <= 0) {
    int full = std::max(rq.R, max_resident_ctas / rq.R * rq.R);
    // Pushed copies on the bulk-copy datapath (all-gather(-v), broadcast) are a 1 read : R writes
    // stream, which the memory system serves fastest with fewer than all SMs writing.  How many
    // depends on the individual GPU (which SMs a grid smaller than the SM count leaves idle follows
    // the chip's own SM layout): of two B200s one ran the 8 x 64 MiB all-gather in 101 us with 136
    // CTAs and 102 with 128, the other in 113 us with 136 and 102-104 with 128 (144: 106 and 110).
    // pl_comm_tune measures it; untuned, 87 % of the resident CTAs (128 of 148) is the safe choice.
    if (p.datapath == PL_DP_TMA && (rq.coll == PL_ALLGATHER || rq.coll == PL_ALLGATHERV || rq.coll == PL_BROADCAST) &&
        rq.algo == PL_ALGO_DIRECT && !rq.staged) {
      const bool one_per_sm = rq.sm_count > 0 && max_resident_ctas == rq.sm_count;
      if (rq.tuned_push_ctas > 0 && rq.tuned_push_ctas <= max_resident_ctas) {
        full = std::max(rq.R, rq.tuned_push_ctas / rq.R * rq.R);
        if (p.idle_count == 0 && one_per_sm && rq.tuned_idle_count > 0 && full + rq.tuned_idle_count == rq.sm_count) {
          p.idle_first = rq.tuned_idle_first;
          p.idle_count = rq.tuned_idle_count;
        }
      } else {
        full = std::max(rq.R, (max_resident_ctas * 87 / 100) / rq.R * rq.R);
        // Untuned: WHICH SMs sit out matters as much as how many (pl_comm_tune); a window of idle
        // SMs that starts at SM 8 was among the fast ones on every B200 tried (97-100 us for the
        // 8 x 64 MiB all-gather), the SMs a plain launch leaves idle were not (98-107 us).
        if (p.idle_count == 0 && one_per_sm && rq.sm_count == 148 && full < rq.sm_count) {
          p.idle_first = 8;
          p.idle_count = rq.sm_count - full;
        }
      }
    }
    // bytes a rank produces in its busiest phase
    uint64_t per_rank = msg;
    if (rq.coll == PL_REDUCE_SCATTER || rq.coll == PL_REDUCE_SCATTERV) per_rank = msg / rq.R;
    if (rq.coll == PL_ALLREDUCE && rq.algo == PL_ALGO_DIRECT_FUSED) per_rank = msg / rq.R;
    uint64_t unit = p.slice_bytes;
    if (unit == 0) unit = std::min<uint64_t>(p.max_slice, std::max<uint64_t>(p.min_slice, per_rank / (full / rq.R)));
    uint64_t want = std::max<uint64_t>(1, (per_rank + unit - 1) / unit) * rq.R;
    p.n_ctas = (int)std::min<uint64_t>(full, std::max<uint64_t>(rq.R, want));
  }
  p.n_ctas = std::max(rq.R, p.n_ctas / rq.R * rq.R);
  // a window of idle SMs goes with a grid of exactly the other SMs
  if (p.idle_count > 0 && (rq.sm_count <= 0 || p.n_ctas + p.idle_count != rq.sm_count)) p.idle_count = 0;
  return p;
}

namespace {
pl_status_t lower_collective(const BuildRequest& rq, Lowered* L, std::string* err);

// Processing phase (PL_HOOK_*): mark the reduce ops that write final output, give their
// destinations the output type, size the second operand.  Only collectives whose outputs are
// written by reduce ops alone qualify: a result that is copied on cannot differ per rank.
pl_status_t apply_hooks(const BuildRequest& rq, Lowered* L, std::string* err) {
  auto fail = [&](pl_status_t st, const char* m) {
    if (err) *err = m;
    return st;
  };
  const int es = elem_size(rq.dtype);
  if (rq.dtype != PL_BF16 && rq.dtype != PL_F32) return fail(PL_ERR_UNSUPPORTED, "processing hooks need a float element type");
  if ((rq.hook & PL_HOOK_F32_OUT) && rq.dtype != PL_BF16) return fail(PL_ERR_UNSUPPORTED, "fp32 output is for bf16 schedules");
  if (rq.packet_ctas_per_rank > 0) return fail(PL_ERR_UNSUPPORTED, "processing hooks are not offered on the packet datapath");
  for (const HostOp& op : L->ops) {
    bool touches_out = op.kind == PL_OP_COPY && op.dst.buf == PL_BUF_OUT;
    for (const pl_ref_t& s : op.src) touches_out = touches_out || s.buf == PL_BUF_OUT;
    if (touches_out)
      return fail(PL_ERR_UNSUPPORTED, "processing hooks need a collective whose outputs are written by its reduce ops only "
                                      "(reduce-scatter, one-shot or fused all-reduce, rooted reduce)");
  }
  const bool f32 = rq.hook & PL_HOOK_F32_OUT;
  for (HostOp& op : L->ops) {
    if (op.dst.buf != PL_BUF_OUT) continue;
    if (op.dst.dtype != rq.dtype) return fail(PL_ERR_UNSUPPORTED, "an op writes non-element-typed output");
    op.final_hook = true;
    if (f32) {
      op.dst.dtype = PL_F32;
      op.dst.offset = op.dst.offset / es * 4;
    }
  }
  for (int r = 0; r < rq.R; ++r) {
    if (rq.hook & PL_HOOK_RESIDUAL) L->aux_bytes[r] = L->out_bytes[r];  // element-typed, laid out like the output
    if (f32) L->out_bytes[r] = L->out_bytes[r] / es * 4;
  }
  return PL_OK;
}
}  // namespace

pl_status_t lower(const BuildRequest& rq, Lowered* L, std::string* err) {
  pl_status_t st = lower_collective(rq, L, err);
  if (st == PL_OK && rq.hook) st = apply_hooks(rq, L, err);
  if (st == PL_OK && rq.stage_ahead) {
    if (!rq.staged) {
      if (err) *err = "PL_OPT_STAGE_AHEAD needs PL_OPT_STAGED";
      return PL_ERR_INVALID_ARG;
    }
    // Stage ops that wait for nothing read only the caller's input and write only staging memory:
    // with two staging buffers they may run while the previous execute still drains.
    for (HostOp& op : L->ops)
      op.stage_ahead = op.kind == PL_OP_COPY && !op.bcast && op.waits.empty() && op.dst.buf == PL_BUF_SCRATCH &&
                       op.src.size() == 1 && op.src[0].buf == PL_BUF_IN;
    L->double_buffered = true;
  }
  return st;
}

namespace {
pl_status_t lower_collective(const BuildRequest& rq, Lowered* L, std::string* err) {
  const int R = rq.R, dt = rq.dtype, es = elem_size(dt);
  auto fail = [&](pl_status_t st, const char* m) {
    if (err) *err = m;
    return st;
  };
  if (R < 2 || R > PL_MAX_RANKS) return fail(PL_ERR_INVALID_ARG, "R out of range");
  if (rq.chunk_bytes == 0 || rq.chunk_bytes % 16) return fail(PL_ERR_INVALID_ARG, "chunk_bytes must be a positive multiple of 16");
  const bool reduces = rq.coll == PL_ALLREDUCE || rq.coll == PL_REDUCE_SCATTER || rq.coll == PL_REDUCE;
  if (reduces && dt == PL_U8) return fail(PL_ERR_UNSUPPORTED, "bytes cannot be reduced");
  Emitter em{L, rq.pol.slice_bytes};
  em.dtype = dt;
  em.min_slice = rq.pol.min_slice;
  em.max_slice = rq.pol.max_slice;
  em.op_overhead_us = rq.pol.datapath == PL_DP_TMA ? 0.2 : 1.5;
  em.wait_overhead_us = rq.pol.datapath == PL_DP_TMA ? 1.5 : 0.5;  // measured on ring schedules
  em.queues_per_rank = std::max(1, rq.pol.n_ctas / R);
  auto two_stages = [&]() { return std::max<uint32_t>(2048, 2 * (rq.pol.stage_bytes / (uint32_t)R) / 128 * 128); };
  L->n_layers = 1;

  if (rq.coll == PL_ALLGATHERV || rq.coll == PL_REDUCE_SCATTERV) {
    if (rq.algo != PL_ALGO_DIRECT) return fail(PL_ERR_UNSUPPORTED, "V collectives are direct only");
    if (rq.staged) return fail(PL_ERR_UNSUPPORTED, "staging is offered for the four fixed-size direct collectives");
    if (!rq.counts_v) return fail(PL_ERR_INVALID_ARG, "sizes missing");
    if (rq.coll == PL_REDUCE_SCATTERV && dt == PL_U8) return fail(PL_ERR_UNSUPPORTED, "bytes cannot be reduced");
    uint64_t total = 0;
    for (int k = 0; k < R; ++k) {
      if ((rq.counts_v[k] * es) % 16) return fail(PL_ERR_ALIGNMENT, "every partition must be a multiple of 16 bytes");
      total += rq.counts_v[k] * es;
    }
    for (int r = 0; r < R; ++r) {
      L->in_bytes[r] = rq.coll == PL_ALLGATHERV ? rq.counts_v[r] * es : total;
      L->out_bytes[r] = rq.coll == PL_ALLGATHERV ? total : rq.counts_v[r] * es;
    }
    L->message_bytes = total;
    em.phase_chunks = 0;
    if (rq.coll == PL_ALLGATHERV) agv_direct(em, R, dt, rq.counts_v, rq.chunk_bytes);
    else rsv_direct(em, R, dt, rq.counts_v, rq.chunk_bytes);
    return PL_OK;
  }
  if (rq.coll == PL_ALLTOALLV) {
    if (rq.algo != PL_ALGO_DIRECT) return fail(PL_ERR_UNSUPPORTED, "all-to-all-v is direct only");
    if (!rq.counts_v) return fail(PL_ERR_INVALID_ARG, "counts missing");
    uint64_t total = 0;
    for (int i = 0; i < R * R; ++i) {
      if ((rq.counts_v[i] * es) % 16) return fail(PL_ERR_ALIGNMENT, "every (src,dst) segment must be a multiple of 16 bytes");
      total += rq.counts_v[i] * es;
    }
    for (int p = 0; p < R; ++p)
      for (int r = 0; r < R; ++r) {
        L->in_bytes[p] += rq.counts_v[p * R + r] * es;
        L->out_bytes[r] += rq.counts_v[p * R + r] * es;
      }
    L->message_bytes = total / R;
    em.phase_chunks = 0;
    if (rq.pol.datapath == PL_DP_TMA) em.stream_slice = 32768;
    a2av_direct(em, R, dt, rq.counts_v, rq.chunk_bytes);
    return PL_OK;
  }
  if (rq.counts_v) return fail(PL_ERR_INVALID_ARG, "counts only apply to all-to-all-v");
  const uint64_t n = rq.count_per_rank;
  if (n == 0) return fail(PL_ERR_INVALID_ARG, "count_per_rank is zero");
  const uint64_t bytes = n * es;

  if (rq.staged && (rq.n_layers > 0 || rq.coll == PL_ALLTOALLV)) return fail(PL_ERR_UNSUPPORTED, "staging is offered for the four fixed-size direct collectives");
  if (rq.n_layers > 0) {
    if (rq.coll != PL_ALLREDUCE) return fail(PL_ERR_UNSUPPORTED, "layered schedules are all-reduce only");
    if (rq.algo != PL_ALGO_ONESHOT && rq.algo != PL_ALGO_DIRECT && rq.algo != PL_ALGO_DIRECT_FUSED)
      return fail(PL_ERR_UNSUPPORTED, "layered schedules support one-shot, direct and direct-fused");
  }
  const int n_layers = std::max(1, rq.n_layers);
  L->n_layers = n_layers;

  if (rq.coll == PL_BROADCAST || rq.coll == PL_REDUCE || rq.coll == PL_SCATTER || rq.coll == PL_GATHER) {
    if (rq.algo != PL_ALGO_DIRECT || rq.staged || rq.n_layers > 0) return fail(PL_ERR_UNSUPPORTED, "rooted collectives are direct, unstaged, single layer");
    if (rq.root < 0 || rq.root >= R) return fail(PL_ERR_INVALID_ARG, "root out of range");
    const int root = rq.root;
    if (rq.coll == PL_BROADCAST || rq.coll == PL_REDUCE) {
      if (bytes % (16 * R)) return fail(PL_ERR_INVALID_ARG, "message bytes must be divisible by 16*R");
      Geo g = make_geo(R, dt, n, n / R, rq.chunk_bytes);
      L->message_bytes = bytes;
      for (int r = 0; r < R; ++r) {
        L->in_bytes[r] = rq.coll == PL_BROADCAST ? (r == root ? bytes : 0) : bytes;
        L->out_bytes[r] = rq.coll == PL_BROADCAST ? bytes : (r == root ? bytes : 0);
      }
      if (rq.coll == PL_BROADCAST) broadcast_composed(em, g, root);
      else {
        if (rq.pol.datapath == PL_DP_TMA && R == 8 && dt == PL_BF16 && bytes >= (64ull << 20)) em.reduce_slice = two_stages();
        reduce_composed(em, g, root);
      }
    } else {
      if (bytes % 16) return fail(PL_ERR_INVALID_ARG, "partition bytes must be a multiple of 16");
      Geo g = make_geo(R, dt, n * R, n, rq.chunk_bytes);
      L->message_bytes = bytes * R;
      for (int r = 0; r < R; ++r) {
        L->in_bytes[r] = rq.coll == PL_SCATTER ? (r == root ? bytes * R : 0) : bytes;
        L->out_bytes[r] = rq.coll == PL_SCATTER ? bytes : (r == root ? bytes * R : 0);
      }
      if (rq.coll == PL_SCATTER) scatter_direct(em, g, root);
      else gather_direct(em, g, root);
    }
    return PL_OK;
  }
  switch (rq.coll) {
    case PL_ALLGATHER: {
      if (bytes % 16) return fail(PL_ERR_INVALID_ARG, "all-gather contribution must be a multiple of 16 bytes");
      Geo g = make_geo(R, dt, n * R, n, rq.chunk_bytes);
      for (int r = 0; r < R; ++r) { L->in_bytes[r] = bytes; L->out_bytes[r] = bytes * R; }
      L->message_bytes = bytes * R;
      if (rq.staged && rq.algo != PL_ALGO_DIRECT) return fail(PL_ERR_UNSUPPORTED, "staged schedules are direct only");
      if (rq.staged) ag_direct_staged(em, g, rq.staging_bytes);
      else if (rq.algo == PL_ALGO_DIRECT) {
        // A push on both datapaths: rank p reads each chunk of its contribution once and writes
        // it into all R outputs.  Register path (working set in L2), R = 8: 8 MiB gathered per rank
        // 19.9 -> 12.0 us against the pull, 1 MiB 4.4 -> 3.2 us.  Bulk-copy path (streaming from
        // HBM), 64 MiB gathered per rank: 101 us with 128-136 CTAs (the grid the policy picks for
        // this 1 read : R writes stream) against 104-106 us for the pull with 144 CTAs; with 144
        // CTAs the push takes 112 us, which is why the grid matters.
        ag_direct_push(em, g);
      } else if (rq.algo == PL_ALGO_RING) ag_ring(em, g, false, nullptr);
      else return fail(PL_ERR_UNSUPPORTED, "all-gather supports direct and ring");
      return PL_OK;
    }
    case PL_ALLTOALL: {
      if (bytes % (16 * R)) return fail(PL_ERR_INVALID_ARG, "message bytes must be divisible by 16*R");
      if (rq.algo != PL_ALGO_DIRECT) return fail(PL_ERR_UNSUPPORTED, "all-to-all is direct only");
      Geo g = make_geo(R, dt, n, n / R, rq.chunk_bytes);
      for (int r = 0; r < R; ++r) L->in_bytes[r] = L->out_bytes[r] = bytes;
      L->message_bytes = bytes;
      if (rq.staged) a2a_direct_staged(em, g, rq.staging_bytes);
      else {
        if (rq.pol.datapath == PL_DP_TMA) em.stream_slice = 32768;
        a2a_direct(em, g);
      }
      return PL_OK;
    }
    case PL_REDUCE_SCATTER: {
      if (bytes % (16 * R)) return fail(PL_ERR_INVALID_ARG, "message bytes must be divisible by 16*R");
      Geo g = make_geo(R, dt, n, n / R, rq.chunk_bytes);
      for (int r = 0; r < R; ++r) { L->in_bytes[r] = bytes; L->out_bytes[r] = bytes / R; }
      L->message_bytes = bytes;
      if (rq.staged && rq.algo != PL_ALGO_DIRECT) return fail(PL_ERR_UNSUPPORTED, "staged schedules are direct only");
      if (rq.staged) rs_direct_staged(em, g, rq.staging_bytes);
      else if (rq.algo == PL_ALGO_DIRECT) {
        if (rq.pol.datapath == PL_DP_TMA && R == 8 && dt == PL_BF16 && bytes >= (64ull << 20)) em.reduce_slice = two_stages();
        rs_direct(em, g);
      }
      else if (rq.algo == PL_ALGO_RING) rs_ring(em, g, false, nullptr);
      else return fail(PL_ERR_UNSUPPORTED, "reduce-scatter supports direct and ring");
      return PL_OK;
    }
    case PL_ALLREDUCE: {
      const bool partitioned = rq.algo == PL_ALGO_DIRECT || rq.algo == PL_ALGO_DIRECT_FUSED || rq.algo == PL_ALGO_RING;
      if (partitioned && bytes % (16 * R)) return fail(PL_ERR_INVALID_ARG, "message bytes must be divisible by 16*R");
      if (bytes % 16) return fail(PL_ERR_INVALID_ARG, "message bytes must be a multiple of 16");
      for (int r = 0; r < R; ++r) L->in_bytes[r] = L->out_bytes[r] = bytes * n_layers;
      L->message_bytes = bytes;
      Geo gp = make_geo(R, dt, n, n / R, rq.chunk_bytes);  // partitioned view
      Geo gw = make_geo(R, dt, n, n, rq.chunk_bytes);      // whole-message view
      if (rq.packet_ctas_per_rank > 0) {
        if (rq.n_layers < 1 || rq.algo != PL_ALGO_ONESHOT) return fail(PL_ERR_UNSUPPORTED, "the packet datapath runs layered one-shot all-reduces");
        if ((bytes / 16) % (uint64_t)rq.packet_ctas_per_rank) return fail(PL_ERR_INVALID_ARG, "message vectors must divide evenly over a rank's CTAs");
        ar_oneshot_packets(em, gw, n_layers, rq.packet_ctas_per_rank);
        return PL_OK;
      }
      if (rq.n_layers > 0) {
        LayerEdges le;
        le.pub.assign(R, -1);
        for (int l = 0; l < n_layers; ++l) {
          le.done.assign(R, -1);
          if (l + 1 < n_layers) {
            if (rq.algo == PL_ALGO_DIRECT_FUSED) {
              int f = em.new_flag();
              le.done.assign(R, f);
            } else {
              for (int r = 0; r < R; ++r) le.done[r] = em.new_flag();
            }
          }
          const uint64_t off = (uint64_t)l * bytes;
          if (rq.algo == PL_ALGO_ONESHOT) ar_oneshot(em, gw, l, off, off, &le);
          else if (rq.algo == PL_ALGO_DIRECT) ar_direct(em, gp, l, off, off, &le);
          else ar_fused(em, gp, l, off, off, &le);
          le.pub = le.done;
        }
        return PL_OK;
      }
      if (rq.staged) {
        if (rq.algo != PL_ALGO_DIRECT) return fail(PL_ERR_UNSUPPORTED, "staged schedules are direct only");
        ar_direct_staged(em, gp, rq.staging_bytes);
        return PL_OK;
      }
      switch (rq.algo) {
        case PL_ALGO_ONESHOT: ar_oneshot(em, gw, 0, 0, 0, nullptr); return PL_OK;
        case PL_ALGO_DIRECT: ar_direct(em, gp, 0, 0, 0, nullptr); return PL_OK;
        case PL_ALGO_DIRECT_FUSED:
          if (rq.pol.datapath == PL_DP_TMA) em.fused_slice = std::max<uint32_t>(2048, 2 * (rq.pol.stage_bytes / (uint32_t)R) / 128 * 128);
          ar_fused(em, gp, 0, 0, 0, nullptr);
          return PL_OK;
        case PL_ALGO_RING: {
          std::vector<int> fin;
          rs_ring(em, gp, true, &fin);
          ag_ring(em, gp, true, &fin);
          return PL_OK;
        }
        case PL_ALGO_TREE: ar_tree(em, gw); return PL_OK;
        default: return fail(PL_ERR_INVALID_ARG, "unknown algorithm");
      }
    }
    default: return fail(PL_ERR_INVALID_ARG, "unknown collective");
  }
}
}  // namespace

// Place ops on queues.  Rank r owns queues {q : q % R == r}; its ops go, in topological
// order, to the least-loaded of its queues (ties to the lowest queue).  Each queue's order is
// therefore a subsequence of the topological order, which is what makes a co-resident grid
// deadlock free: the unfinished op with the smallest topological index is always at the head
// of its queue and all it waits for has already run.
void assign_queues(Lowered* L, int R, int n_queues, bool by_level) {
  const int per_rank = std::max(1, n_queues / R);
  std::vector<uint64_t> load((size_t)per_rank * R, 0);
  // by_level: ops at the same depth of the flag-dependency graph can run at the same time, so
  // a queue takes a second one only when every queue of the rank has one; load breaks ties
  std::vector<int> flag_level(by_level ? L->n_flags : 0, 0);
  std::vector<std::vector<int>> at_level((size_t)per_rank * R);
  L->flag_need.assign(L->n_flags, 0);
  // queue index ranges [lo, hi) inside a rank for each role (role 0 = all of them)
  int lo[4] = {0, 0, 0, 0}, hi[4] = {per_rank, per_rank, per_rank, per_rank};
  if (L->role_queues[1] + L->role_queues[2] + L->role_queues[3] == per_rank) {
    int at = 0;
    for (int i = 1; i < 4; ++i) {
      lo[i] = at;
      at += L->role_queues[i];
      hi[i] = at;
    }
  }
  int topo = 0;
  for (HostOp& op : L->ops) {
    op.topo = topo++;
    uint64_t cost = op.count * elem_size(op.dst.dtype) * (op.bcast ? R : 1);
    for (const pl_ref_t& s : op.src) cost += op.count * elem_size(s.dtype);
    cost += 2048;  // fixed per-op overhead so that many tiny ops still spread out
    const int role = (op.role >= 0 && op.role < 4 && hi[op.role] > lo[op.role]) ? op.role : 0;
    int lv = 0;
    if (by_level) {
      for (int w : op.waits) lv = std::max(lv, flag_level[w]);
      for (int sgn : {op.signal, op.signal2})
        if (sgn >= 0) flag_level[sgn] = std::max(flag_level[sgn], lv + 1);
    }
    auto key = [&](int j) {
      const size_t q = (size_t)j * R + op.exec_rank;
      const uint64_t same = by_level && (int)at_level[q].size() > lv ? (uint64_t)at_level[q][lv] : 0;
      return std::make_pair(same, load[q]);
    };
    int best = lo[role];
    if (L->queues_preassigned) {
      best = op.queue / R;
    } else {
      for (int j = lo[role] + 1; j < hi[role]; ++j)
        if (key(j) < key(best)) best = j;
    }
    load[(size_t)best * R + op.exec_rank] += cost;
    if (by_level) {
      std::vector<int>& al = at_level[(size_t)best * R + op.exec_rank];
      if ((int)al.size() <= lv) al.resize(lv + 1, 0);
      al[lv] += 1;
    }
    op.queue = best * R + op.exec_rank;
    if (op.signal >= 0) L->flag_need[op.signal] += 1;
    if (op.signal2 >= 0) L->flag_need[op.signal2] += 1;
  }
}

int level_width(const Lowered& L, int R) {
  // level of an op = length of the longest chain of flag edges that ends in it
  std::vector<int> flag_level(L.n_flags, 0);
  std::vector<std::vector<int>> width(R);
  int best = 1;
  for (const HostOp& op : L.ops) {
    int lv = 0;
    for (int w : op.waits) lv = std::max(lv, flag_level[w]);
    for (int sgn : {op.signal, op.signal2})
      if (sgn >= 0) flag_level[sgn] = std::max(flag_level[sgn], lv + 1);
    std::vector<int>& wr = width[op.exec_rank];
    if ((int)wr.size() <= lv) wr.resize(lv + 1, 0);
    best = std::max(best, ++wr[lv]);
  }
  return best;
}

namespace {
using Key = std::pair<int, int>;  // (buf kind, rank)
}  // namespace

pl_status_t validate(const Lowered& L, int R, std::string* err, bool bulk_datapath) {
  char msg[256];
  auto fail = [&](const char* m) {
    if (err) *err = m;
    return PL_ERR_INVALID_SCHEDULE;
  };
  const size_t n = L.ops.size();
  // 1. topological sanity: each flag's signals all come from ops before any waiter
  std::vector<int> last_signal(L.n_flags, -1), first_wait(L.n_flags, INT32_MAX);
  std::vector<uint32_t> need(L.n_flags, 0);
  for (size_t i = 0; i < n; ++i) {
    const HostOp& op = L.ops[i];
    if (op.topo != (int)i) return fail("ops are not stored in topological order");
    for (int s : {op.signal, op.signal2})
      if (s >= 0) {
        if (s >= L.n_flags) return fail("signal flag out of range");
        last_signal[s] = std::max(last_signal[s], (int)i);
        need[s]++;
      }
    if (op.signal >= 0 && op.signal == op.signal2) return fail("op signals the same flag twice");
    if (op.waits.size() > PL_MAX_WAITS) return fail("too many waits on one op");
    if (op.src.size() > PL_MAX_SRC || op.src.empty()) return fail("bad source count");
    for (int w : op.waits) {
      if (w < 0 || w >= L.n_flags) return fail("wait flag out of range");
      first_wait[w] = std::min(first_wait[w], (int)i);
    }
  }
  for (int f = 0; f < L.n_flags; ++f) {
    if (need[f] != L.flag_need[f]) return fail("flag_need does not match the number of signals");
    if (first_wait[f] != INT32_MAX && need[f] == 0) return fail("a flag is waited on but never signalled");
    if (first_wait[f] != INT32_MAX && last_signal[f] >= first_wait[f]) return fail("a waiter precedes one of its signals in the topological order");
  }
  // 2. queue order embeds in the topological order (ops are appended per queue in topo order
  //    by construction; check exec_rank / queue agreement)
  for (const HostOp& op : L.ops) {
    if (op.queue < 0) return fail("op without a queue");
    if (op.queue % R != op.exec_rank) return fail("op placed on another rank's queue");
  }
  // 3. alignment and bounds
  for (const HostOp& op : L.ops) {
    auto check = [&](const pl_ref_t& r, uint64_t limit_bytes) -> const char* {
      uint64_t b = op.count * elem_size(r.dtype);
      if (r.offset % 16 || b % 16) return "operand not 16-byte aligned";
      if (r.rank < 0 || r.rank >= R) return "rank out of range";
      if (r.offset + b > limit_bytes) return "operand exceeds its buffer";
      return nullptr;
    };
    auto limit = [&](const pl_ref_t& r) {
      return r.buf == PL_BUF_IN ? L.in_bytes[r.rank] : r.buf == PL_BUF_OUT ? L.out_bytes[r.rank] : L.scratch_per_rank[r.rank];
    };
    if (op.dst.buf == PL_BUF_IN) return fail("an op writes an input buffer");
    if (op.bcast) {
      if (op.dst.buf != PL_BUF_OUT) return fail("broadcast destination must be an output");
      for (int r = 0; r < R; ++r) {
        pl_ref_t d = op.dst;
        d.rank = r;
        if (const char* m = check(d, L.out_bytes[r])) return fail(m);
      }
    } else if (const char* m = check(op.dst, limit(op.dst))) {
      return fail(m);
    }
    for (const pl_ref_t& s : op.src)
      if (const char* m = check(s, limit(s))) return fail(m);
  }
  // 3b. two staging buffers alternated by launch parity: an op that may run while the previous
  //     execute still drains must touch nothing that execute can touch.  The previous execute
  //     reads inputs, writes outputs and uses the OTHER staging buffer and flag set, so an early op
  //     may only read the caller's input, write staging memory and signal; it cannot wait (its
  //     flag set belongs to this execute, whose other ops have not started).
  for (const HostOp& op : L.ops) {
    if (!op.stage_ahead) continue;
    if (!L.double_buffered) return fail("an op is marked for early staging in a schedule with one staging buffer");
    if (!op.waits.empty()) return fail("an early stage op waits on a flag");
    if (op.kind != PL_OP_COPY || op.bcast || op.dst.buf != PL_BUF_SCRATCH) return fail("an early stage op writes something other than staging memory");
    for (const pl_ref_t& s : op.src)
      if (s.buf != PL_BUF_IN) return fail("an early stage op reads something other than the caller's input");
  }
  // 4. memory hazards, replayed in topological order over a map of disjoint segments per
  //    buffer.  Outputs: every byte written exactly once and fully covered.  Scratch (staging
  //    slots may be reused within one execute): a write must happen after the previous write
  //    of those bytes and after every read of that previous version.  Every read of bytes the
  //    schedule writes must happen after that write.  "Happens after" = reachable through
  //    wait edges (a wait on a flag orders the waiter after ALL of the flag's signallers) or
  //    program order on one queue.
  std::vector<std::vector<int>> signallers(L.n_flags);
  for (size_t i = 0; i < n; ++i)
    for (int f : {L.ops[i].signal, L.ops[i].signal2})
      if (f >= 0) signallers[f].push_back((int)i);
  std::vector<int> stamp(n, -1);
  int query = 0;
  // What program order on one queue is worth depends on the executor.  The register executor
  // puts a CTA-wide barrier between ops: everything of op a is done before anything of a later
  // op on its queue.  The bulk-copy executor runs ahead: its producer warp issues the loads of
  // later ops while the consumer warps (register stores) and the copier warp (bulk stores) are
  // still writing earlier ones, and those two kinds of writers do not wait for each other.
  // There, on one queue: a later op's READ is never ordered after an earlier op's write; an
  // earlier op's reads are complete before a later op stores or signals (the ring is consumed
  // in order); an earlier op's WRITES are complete before a later op's stores or signal only
  // if both leave through the same kind of writer.
  auto writer_class = [&](const HostOp& o) {  // 0: consumer warps, 1: copier warp (bulk stores)
    if (o.kind == PL_OP_COPY) return 1;
    bool plain = true;
    for (const pl_ref_t& r : o.src)
      if (r.dtype != o.dst.dtype) plain = false;
    return (o.bcast && plain && !o.final_hook) ? 1 : 0;
  };
  // a_writes: the access of op a that must be complete is a write (else a read);
  // x_reads: the access of op x that must come later is a read (else a write).
  auto happens_before = [&](int a, int x, bool a_writes, bool x_reads) -> bool {
    if (a >= x) return false;
    ++query;
    std::vector<std::pair<int, int>> stack{{x, 0}};
    stamp[x] = query;
    size_t visited = 0;
    const HostOp& oa = L.ops[a];
    while (!stack.empty()) {
      auto [y, depth] = stack.back();
      stack.pop_back();
      const HostOp& oy = L.ops[y];
      if (oy.queue == oa.queue && a < y) {
        if (!bulk_datapath) return true;
        const bool same_writer = writer_class(oa) == writer_class(oy);
        if (y == x) {
          if (!x_reads && (!a_writes || same_writer)) return true;
        } else if (!a_writes || same_writer) {
          return true;  // y's signal is released after a's access is complete
        }
      }
      if (depth >= 6 || ++visited > 200000) continue;
      for (int f : oy.waits)
        for (int sgn : signallers[f]) {
          if (sgn == a) return true;
          if (sgn > a && stamp[sgn] != query) {
            stamp[sgn] = query;
            stack.push_back({sgn, depth + 1});
          }
        }
    }
    return false;
  };
  struct Seg {
    uint64_t hi;
    int writer;
    std::vector<int> readers;
  };
  std::map<Key, std::map<uint64_t, Seg>> mem;
  // split so that `at` is a segment boundary
  auto split = [](std::map<uint64_t, Seg>& m, uint64_t at) {
    auto it = m.upper_bound(at);
    if (it == m.begin()) return;
    --it;
    if (it->first < at && at < it->second.hi) {
      Seg right = it->second;
      it->second.hi = at;
      m[at] = right;
    }
  };
  for (size_t i = 0; i < n; ++i) {
    const HostOp& op = L.ops[i];
    for (const pl_ref_t& src : op.src) {
      auto mit = mem.find({src.buf, src.rank});
      if (mit == mem.end()) continue;
      auto& m = mit->second;
      const uint64_t lo = src.offset, hi = src.offset + op.count * elem_size(src.dtype);
      auto it = m.upper_bound(lo);
      if (it != m.begin()) --it;
      for (; it != m.end() && it->first < hi; ++it) {
        if (it->second.hi <= lo) continue;
        const int w = it->second.writer;
        bool direct = false;
        for (int f : op.waits)
          if (f == L.ops[w].signal || f == L.ops[w].signal2) direct = true;
        if (!direct && !happens_before(w, (int)i, true, true)) {
          std::snprintf(msg, sizeof msg, "op %zu reads bytes written by op %d without being ordered after it", i, w);
          return fail(msg);
        }
        if (src.buf == PL_BUF_SCRATCH) it->second.readers.push_back((int)i);
      }
    }
    const uint64_t b = op.count * elem_size(op.dst.dtype);
    for (int r = 0; r < R; ++r) {
      if (!op.bcast && r != op.dst.rank) continue;
      auto& m = mem[{op.dst.buf, r}];
      const uint64_t lo = op.dst.offset, hi = lo + b;
      split(m, lo);
      split(m, hi);
      auto it = m.lower_bound(lo);
      while (it != m.end() && it->first < hi) {
        if (op.dst.buf == PL_BUF_OUT) {
          std::snprintf(msg, sizeof msg, "ops %d and %zu write overlapping bytes of the output of rank %d", it->second.writer, i, r);
          return fail(msg);
        }
        if (!happens_before(it->second.writer, (int)i, true, false)) {
          std::snprintf(msg, sizeof msg, "op %zu overwrites scratch written by op %d without being ordered after it", i, it->second.writer);
          return fail(msg);
        }
        for (int rd : it->second.readers)
          if (rd != (int)i && !happens_before(rd, (int)i, false, false)) {
            std::snprintf(msg, sizeof msg, "op %zu overwrites scratch that op %d may still be reading", i, rd);
            return fail(msg);
          }
        it = m.erase(it);
      }
      m[lo] = Seg{hi, (int)i, {}};
    }
  }
  for (int r = 0; r < R; ++r) {
    uint64_t covered = 0;
    auto mit = mem.find({PL_BUF_OUT, r});
    if (mit != mem.end())
      for (const auto& kv : mit->second) {
        if (kv.first != covered) break;
        covered = kv.second.hi;
      }
    if (covered != L.out_bytes[r]) {
      std::snprintf(msg, sizeof msg, "output of rank %d is covered up to byte %llu of %llu", r,
                    (unsigned long long)covered, (unsigned long long)L.out_bytes[r]);
      return fail(msg);
    }
  }
  return PL_OK;
}

}  // namespace pl
