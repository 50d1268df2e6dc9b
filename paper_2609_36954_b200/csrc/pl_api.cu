// C-ABI layer: handles, argument checks, device upload of a lowered schedule, launches.
#include <cuda_runtime.h>

#include <algorithm>
#include <atomic>
#include <cstdio>
#include <cstring>
#include <mutex>
#include <new>
#include <string>
#include <vector>

#include "pl_api_internal.h"
#include "pl_internal.h"
#include "pl_kernels.h"

using namespace pl;

namespace pl {
std::atomic<uint64_t> g_launches{0};

bool on_comm_device(pl_comm_s* comm) {
  if (comm->planner) return true;
  int d = -1;
  if (cudaGetDevice(&d) != cudaSuccess) { cudaGetLastError(); return false; }
  if (d != comm->device) {
    comm->last_error = "the current CUDA device is not the communicator's";
    return false;
  }
  return true;
}
}  // namespace pl

struct pl_schedule_s {
  pl_comm_t comm = nullptr;
  Lowered L;
  Policy pol{};
  pl_sched_info_t info{};
  uint64_t timeout_ns = 0;
  bool no_l2_hints = false;
  bool sm_window = false;         // launch one CTA per SM; the SMs outside sm_mask sit out (pol.idle_first / idle_count)
  uint32_t sm_mask[5] = {0, 0, 0, 0, 0};
  size_t off_sm_state = 0;
  bool inputs_last_use = false;   // PL_OPT_INPUTS_LAST_USE asked for and every input byte is read once
  bool trace = false;
  bool overlap_launch = false;
  bool bcast_copies = false;      // some COPY op writes every rank's output
  bool pipelined_reduce = false;  // bulk-copy datapath: every reduce op is plain, run the 12-warp variant
  bool stage_ahead = false;       // double-buffered staging: two scratch halves and flag sets, chosen by launch parity
  uint64_t scratch_half = 0;      // bytes of one half (all ranks)
  int packet_ctas_per_rank = 0;   // > 0: packet datapath (layered one-shot all-reduce), CTAs per rank
  long long packet_break_op = -1; // test hook (pl_schedule_debug_break_wait on a packet schedule)
  size_t off_trace = 0;
  float out_scale = 1.0f;
  uint32_t hook = 0;  // PL_HOOK_* bits
  // host copies in device (queue-major) order
  std::vector<DevOp> dev_ops;
  std::vector<uint64_t> srcs;
  std::vector<DevWait> waits;
  std::vector<int> topo_to_dev;  // topological index -> position in dev_ops
  uint32_t src_stride = 1, wait_stride = 1;
  // device
  char* d_blob = nullptr;
  size_t blob_bytes = 0;
  size_t off_ops = 0, off_srcs = 0, off_waits = 0, off_flags = 0, off_epoch = 0;
  size_t sync_bytes = 0;  // flags + epoch, zeroed at build and by reset
  char* d_scratch = nullptr;
  uint64_t scratch_off[PL_MAX_RANKS] = {0};
  uint64_t scratch_total = 0;
};

namespace {

size_t align_up(size_t x, size_t a) { return (x + a - 1) / a * a; }

uint64_t pack(const pl_schedule_s& S, const pl_ref_t& r) {
  int slot = r.buf == PL_BUF_IN ? kSlotIn + r.rank : r.buf == PL_BUF_OUT ? kSlotOut + r.rank : kSlotScratch + r.rank;
  return ((uint64_t)slot << 48) | r.offset;
}

void fill_info(pl_schedule_s* S, int R) {
  pl_sched_info_t& I = S->info;
  std::memset(&I, 0, sizeof(I));
  const Lowered& L = S->L;
  I.n_ops = L.ops.size();
  I.n_queues = S->pol.n_ctas;
  I.n_flags = L.n_flags;
  I.n_layers = L.n_layers;
  for (const HostOp& op : L.ops) {
    I.n_waits += op.waits.size();
    for (const pl_ref_t& s : op.src) I.bytes_read += op.count * elem_size(s.dtype);
    I.bytes_written += op.count * elem_size(op.dst.dtype) * (op.bcast ? R : 1);
    if (op.final_hook && (S->hook & PL_HOOK_RESIDUAL)) I.bytes_read += op.count * elem_size(S->comm->dtype) * (op.bcast ? R : 1);
  }
  I.message_bytes = L.message_bytes;
  for (int r = 0; r < R; ++r) {
    I.scratch_bytes += L.scratch_per_rank[r] * (S->stage_ahead ? 2 : 1);
    I.in_bytes[r] = L.in_bytes[r];
    I.out_bytes[r] = L.out_bytes[r];
    I.aux_bytes[r] = L.aux_bytes[r];
  }
  // Compulsory traffic: what the ops read from the caller's inputs counts once per byte (the union
  // of the ranges per rank), what they read from outputs or scratch was produced by this launch
  // and counts every time, like every write.
  {
    std::vector<std::vector<std::pair<uint64_t, uint64_t>>> ranges(R);
    uint64_t other_reads = 0;
    for (const HostOp& op : L.ops)
      for (const pl_ref_t& s : op.src) {
        const uint64_t b = op.count * elem_size(s.dtype);
        if (s.buf == PL_BUF_IN) ranges[s.rank].emplace_back(s.offset, s.offset + b);
        else other_reads += b;
      }
    uint64_t in_once = 0, in_reads = 0;
    for (const auto& v : ranges)
      for (const auto& iv : v) in_reads += iv.second - iv.first;
    for (auto& v : ranges) {
      std::sort(v.begin(), v.end());
      uint64_t hi = 0;
      for (const auto& iv : v) {
        if (iv.second <= hi) continue;
        in_once += iv.second - std::max(iv.first, hi);
        hi = iv.second;
      }
    }
    uint64_t aux_reads = 0;
    for (int r = 0; r < R; ++r) aux_reads += L.aux_bytes[r];
    I.hbm_bytes = in_once + other_reads + aux_reads + I.bytes_written;
    if (in_reads != in_once) S->inputs_last_use = false;  // some input byte is read more than once
  }
  I.out_dtype = (S->hook & PL_HOOK_F32_OUT) ? PL_F32 : S->comm->dtype;
  I.hook = S->hook;
  I.grid = S->pol.n_ctas;
  I.idle_sm_first = S->sm_window ? S->pol.idle_first : 0;
  I.idle_sm_count = S->sm_window ? S->pol.idle_count : 0;
  I.threads = S->pol.threads;
  I.smem_bytes = S->pol.datapath == PL_DP_TMA ? (int32_t)exec_tma_smem_bytes(S->pol.stages, S->pol.stage_bytes) : 0;
  I.datapath = S->pol.datapath;
  I.stages = S->pol.stages;
  I.stage_bytes = S->pol.stage_bytes;
  I.slice_bytes = S->pol.slice_bytes;
}

// Flatten the lowered ops into the device arrays (host side): op i of queue q at index
// i * n_queues + q, queues padded to the longest one, empty queues get one placeholder.
void flatten(pl_schedule_s* S, int dtype) {
  const Lowered& L = S->L;
  const int nq = S->pol.n_ctas;
  size_t max_src = 1, max_wait = 1;
  std::vector<uint32_t> qlen(nq, 0);
  for (const HostOp& op : L.ops) {
    max_src = std::max(max_src, op.src.size());
    max_wait = std::max(max_wait, op.waits.size());
    qlen[op.queue]++;
  }
  S->src_stride = (uint32_t)max_src;
  S->wait_stride = (uint32_t)max_wait;
  uint32_t max_len = 1;
  for (int q = 0; q < nq; ++q) max_len = std::max(max_len, qlen[q]);
  const size_t n = (size_t)max_len * nq;
  DevOp nop{};
  nop.kind = kNopKind;
  nop.signal = nop.signal2 = kNoFlag;
  S->dev_ops.assign(n, nop);
  S->srcs.assign(n * max_src, 0);
  S->waits.assign(n * max_wait, DevWait{0, 0});
  S->topo_to_dev.assign(L.ops.size(), 0);
  std::vector<uint32_t> cursor(nq, 0);
  for (const HostOp& op : L.ops) {  // topological order => per-queue order is a subsequence
    const uint32_t i = cursor[op.queue]++;
    const size_t pos = (size_t)i * nq + op.queue;
    S->topo_to_dev[op.topo] = (int)pos;
    DevOp& d = S->dev_ops[pos];
    d.kind = op.kind;
    d.n_src = (uint32_t)op.src.size();
    d.remaining = qlen[op.queue] - 1 - i;
    d.n_wait = (uint32_t)op.waits.size();
    d.signal = op.signal >= 0 ? (uint32_t)op.signal : kNoFlag;
    d.signal2 = op.signal2 >= 0 ? (uint32_t)op.signal2 : kNoFlag;
    d.flags = (op.bcast ? kDstBcast : 0u) | ((op.kind != PL_OP_COPY && op.dst.dtype != dtype) ? kDstF32 : 0u) |
              (op.final_hook ? kFinal : 0u) | (op.stage_ahead ? kStageAhead : 0u);
    d.count = op.count;
    d.dst = pack(*S, op.dst);
    d.topo = (uint32_t)op.topo;
    for (size_t k = 0; k < op.src.size(); ++k) {
      S->srcs[pos * max_src + k] = pack(*S, op.src[k]);
      if (op.kind != PL_OP_COPY && op.src[k].dtype != dtype) d.src_f32_mask |= 1u << k;
    }
    for (size_t k = 0; k < op.waits.size(); ++k)
      S->waits[pos * max_wait + k] = DevWait{(uint32_t)op.waits[k], L.flag_need[op.waits[k]]};
  }
}

pl_status_t upload(pl_schedule_s* S, int R) {
  size_t off = 0;
  auto place = [&](size_t bytes) {
    size_t o = off;
    off = align_up(off + std::max<size_t>(bytes, 16), 256);
    return o;
  };
  S->off_ops = place(S->dev_ops.size() * sizeof(DevOp));
  S->off_srcs = place(S->srcs.size() * sizeof(uint64_t));
  S->off_waits = place(S->waits.size() * sizeof(DevWait));
  S->off_flags = place((size_t)std::max(1, S->L.n_flags) * sizeof(unsigned long long) * (S->stage_ahead ? 2 : 1));
  S->off_epoch = place(4 * sizeof(unsigned long long));
  S->off_sm_state = place(3 * sizeof(unsigned long long));   // claim words of SM-window launches (zeroed with the flags)
  S->sync_bytes = off - S->off_flags;
  if (S->trace) S->off_trace = place(2 * S->L.ops.size() * sizeof(unsigned long long));
  S->blob_bytes = off;
  if (cudaMalloc(&S->d_blob, S->blob_bytes) != cudaSuccess) { cudaGetLastError(); return PL_ERR_OOM; }
  std::vector<char> host(S->blob_bytes, 0);
  std::memcpy(host.data() + S->off_ops, S->dev_ops.data(), S->dev_ops.size() * sizeof(DevOp));
  std::memcpy(host.data() + S->off_srcs, S->srcs.data(), S->srcs.size() * sizeof(uint64_t));
  std::memcpy(host.data() + S->off_waits, S->waits.data(), S->waits.size() * sizeof(DevWait));
  if (cudaMemcpy(S->d_blob, host.data(), S->blob_bytes, cudaMemcpyHostToDevice) != cudaSuccess) {
    cudaGetLastError();
    return PL_ERR_CUDA;
  }
  uint64_t total = 0;
  for (int r = 0; r < R; ++r) {
    S->scratch_off[r] = total;
    total += align_up(S->L.scratch_per_rank[r], 256);
  }
  if (S->stage_ahead) {  // second staging buffer of every rank, one half behind the first
    S->scratch_half = total;
    total *= 2;
  }
  S->scratch_total = total;
  if (total) {
    if (cudaMalloc(&S->d_scratch, total) != cudaSuccess) { cudaGetLastError(); return PL_ERR_OOM; }
    // packet buffers: a tag left over from whoever used this memory before must never match
    if (S->packet_ctas_per_rank && cudaMemset(S->d_scratch, 0, total) != cudaSuccess) { cudaGetLastError(); return PL_ERR_CUDA; }
  }
  return PL_OK;
}

// Packet datapath (layered one-shot all-reduce of a small message): pick the CTAs per rank and
// the CTA size, lower, check that all rank groups can be resident at once, upload.
pl_status_t build_packets(pl_comm_t comm, BuildRequest rq, Policy pol, uint64_t timeout, uint32_t flags, float out_scale,
                          pl_schedule_t* out) {
  auto fail = [&](pl_status_t st, const char* m) {
    comm->last_error = m;
    return st;
  };
  const int R = comm->R, es = elem_size(comm->dtype);
  if (rq.n_layers < 1 || rq.coll != PL_ALLREDUCE) return fail(PL_ERR_UNSUPPORTED, "the packet datapath runs layered all-reduces (pl_schedule_build_layers)");
  if (rq.algo != PL_ALGO_ONESHOT) return fail(PL_ERR_UNSUPPORTED, "the packet datapath is one-shot");
  if (comm->dtype == PL_U8) return fail(PL_ERR_UNSUPPORTED, "bytes cannot be reduced");
  if (rq.staged || (flags & PL_OPT_STAGED)) return fail(PL_ERR_UNSUPPORTED, "packets are their own staging");
  const uint64_t bytes = rq.count_per_rank * (uint64_t)es;
  if (bytes == 0 || bytes % 16) return fail(PL_ERR_INVALID_ARG, "message bytes must be a positive multiple of 16");
  const uint64_t units = bytes / 16;
  int G = 0;
  if (pol.n_ctas > 0) {
    G = pol.n_ctas / R;
    if (G * R != pol.n_ctas || (G != 1 && G != 2 && G != 4 && G != 8) || units % (uint64_t)G)
      return fail(PL_ERR_INVALID_ARG, "n_ctas must be R times 1, 2, 4 or 8 and divide the message vectors");
  } else if (bytes <= 4096) {
    // One CTA per rank: the rank's join is a CTA barrier, which does not wait for the output stores
    // to reach L2 as the cluster barrier of a multi-CTA rank must (measured on B200, R = 8, 80
    // layers: 1.78 / 1.82 / 2.05 us per layer at 1 / 2 / 4 KiB against 2.7-2.9 us with two or more
    // CTAs per rank; above 4 KiB the 2 x R x message bytes of packets a single CTA has to read take over).
    G = 1;
  } else {
    for (G = 8; G > 1; G /= 2)
      if (units % (uint64_t)G == 0 && units / (uint64_t)G >= 8) break;
  }
  const uint64_t per_cta = units / (uint64_t)G;
  int threads = pol.threads > 0 ? pol.threads : (int)std::min<uint64_t>(exec_packet_max_threads(), (per_cta + 31) / 32 * 32);
  if (threads > exec_packet_max_threads()) return fail(PL_ERR_INVALID_ARG, "at most 256 threads per CTA on the packet datapath");
  if ((per_cta + threads - 1) / threads > (uint64_t)exec_packet_max_units_per_thread())
    return fail(PL_ERR_UNSUPPORTED, "message too large for the packet datapath (at most 4 vectors per thread)");
  if (!comm->planner) {
    const int groups = exec_packet_max_groups(comm->dtype, G, threads);
    if (groups <= 0) return PL_ERR_CUDA;
    if (groups < R) return fail(PL_ERR_OVERSUBSCRIBED, "the rank groups of the packet datapath cannot all be resident");
  }
  pol.datapath = PL_DP_PACKET;
  pol.n_ctas = G * R;
  pol.threads = threads;
  pol.stages = 0;
  pol.stage_bytes = 0;
  pol.slice_bytes = (uint32_t)(per_cta * 16);
  rq.pol = pol;
  rq.packet_ctas_per_rank = G;
  rq.chunk_bytes = ((uint64_t)1 << 40);

  pl_schedule_s* S = new (std::nothrow) pl_schedule_s();
  if (!S) return PL_ERR_OOM;
  S->comm = comm;
  S->pol = pol;
  S->timeout_ns = timeout;
  S->trace = (flags & PL_OPT_TRACE) != 0;
  S->overlap_launch = (flags & PL_OPT_OVERLAP_LAUNCH) != 0;
  S->out_scale = out_scale;
  S->packet_ctas_per_rank = G;
  std::string err;
  pl_status_t st = lower(rq, &S->L, &err);
  if (st == PL_OK) {
    assign_queues(&S->L, R, pol.n_ctas, false);
    if (!(flags & PL_OPT_SKIP_VALIDATE)) st = validate(S->L, R, &err, false);
  }
  if (st != PL_OK) {
    comm->last_error = err;
    delete S;
    return st;
  }
  fill_info(S, R);
  flatten(S, comm->dtype);
  if (!comm->planner) {
    st = upload(S, R);
    if (st != PL_OK) {
      pl_schedule_destroy(S);
      return st;
    }
  }
  {
    std::lock_guard<std::mutex> g(comm->mu);
    comm->schedules.push_back(S);
  }
  *out = S;
  return PL_OK;
}

pl_status_t build_common(pl_comm_t comm, BuildRequest rq, const pl_sched_opts_t* opts, pl_schedule_t* out) {
  if (!comm || !out) return PL_ERR_INVALID_ARG;
  *out = nullptr;
  if (!on_comm_device(comm)) return PL_ERR_INVALID_ARG;
  Policy pol{};
  uint64_t timeout = 2000000000ull;
  uint32_t flags = 0, hook = 0;
  float out_scale = 1.0f;
  bool idle_asked = false;  // opts name a window of idle SMs
  if (opts) {
    if (opts->struct_size != sizeof(pl_sched_opts_t)) return PL_ERR_INVALID_ARG;
    pol.n_ctas = opts->n_ctas;
    pol.threads = opts->threads;
    pol.datapath = opts->datapath;
    pol.stages = opts->stages;
    pol.stage_bytes = opts->stage_bytes;
    pol.slice_bytes = opts->slice_bytes;
    if (opts->timeout_ns) timeout = opts->timeout_ns;
    flags = opts->flags;
    rq.staged = (flags & PL_OPT_STAGED) != 0;
    rq.staging_bytes = opts->staging_bytes;
    if (opts->out_scale != 0.0f) {
      if (comm->dtype != PL_BF16 && comm->dtype != PL_F32) return PL_ERR_UNSUPPORTED;
      out_scale = opts->out_scale;
    }
    hook = opts->hook;
    if (opts->idle_sm_count < 0 || opts->idle_sm_first < 0) return PL_ERR_INVALID_ARG;
    if (opts->idle_sm_count > 0) {
      // an explicit window: the grid is every other SM
      const int active = comm->sm_count - opts->idle_sm_count;
      if (opts->idle_sm_first + opts->idle_sm_count > comm->sm_count || active < comm->R || active % comm->R) return PL_ERR_INVALID_ARG;
      if (pol.n_ctas != 0 && pol.n_ctas != active) return PL_ERR_INVALID_ARG;
      pol.n_ctas = active;
      pol.idle_first = opts->idle_sm_first;
      pol.idle_count = opts->idle_sm_count;
      idle_asked = true;
    }
    if (hook & ~(PL_HOOK_RESIDUAL | PL_HOOK_F32_OUT)) return PL_ERR_INVALID_ARG;
    if (hook && comm->dtype != PL_BF16 && comm->dtype != PL_F32) return PL_ERR_UNSUPPORTED;
    if (pol.threads < 0 || pol.threads % 32 || pol.threads > exec_max_threads()) return PL_ERR_INVALID_ARG;
    if (pol.n_ctas < 0 || pol.stages < 0 || pol.stage_bytes % 16 || pol.slice_bytes % 16) return PL_ERR_INVALID_ARG;
    if (pol.datapath < PL_DP_AUTO || pol.datapath > PL_DP_PACKET) return PL_ERR_INVALID_ARG;
  }
  rq.R = comm->R;
  rq.dtype = comm->dtype;
  rq.hook = hook;
  rq.stage_ahead = (flags & PL_OPT_STAGE_AHEAD) != 0;
  if (rq.stage_ahead && (!(flags & PL_OPT_STAGED) || !(flags & PL_OPT_OVERLAP_LAUNCH) || (flags & PL_OPT_TRACE) || hook)) {
    comm->last_error = "PL_OPT_STAGE_AHEAD needs PL_OPT_STAGED and PL_OPT_OVERLAP_LAUNCH (and neither trace nor hooks)";
    return PL_ERR_INVALID_ARG;
  }
  if (pol.datapath == PL_DP_PACKET && hook) {
    comm->last_error = "processing hooks are not offered on the packet datapath";
    return PL_ERR_UNSUPPORTED;
  }
  if (pol.datapath == PL_DP_PACKET) return build_packets(comm, rq, pol, timeout, flags, out_scale, out);
  rq.pol = pol;
  rq.tuned_push_ctas = comm->tuned_push_ctas;
  rq.tuned_idle_first = comm->tuned_idle_first;
  rq.tuned_idle_count = comm->tuned_idle_count;
  rq.sm_count = comm->sm_count;
  const int requested = pol.n_ctas;
  pol = default_policy(rq, 0);  // datapath, threads, ring geometry
  rq.pol = pol;
  rq.pol.n_ctas = requested;
  if (pol.datapath == PL_DP_TMA) {
    if (pol.stages < 2 || pol.stages > 8 || pol.stage_bytes < 1024 || exec_tma_smem_bytes(pol.stages, pol.stage_bytes) > 227 * 1024)
      return PL_ERR_INVALID_ARG;
    pol.threads = exec_tma_threads(false);
    rq.pol.threads = pol.threads;
  }
  int capacity = 148 * (pol.datapath == PL_DP_TMA ? 2 : 1);
  if (!comm->planner) {
    int per_sm = pol.datapath == PL_DP_TMA ? exec_tma_max_ctas_per_sm(comm->dtype, pol.stages, pol.stage_bytes)
                                           : exec_max_ctas_per_sm(comm->dtype, pol.threads);
    if (per_sm <= 0) return PL_ERR_CUDA;
    capacity = per_sm * comm->sm_count;
  }
  pol = default_policy(rq, capacity);
  if (requested > capacity) return PL_ERR_OVERSUBSCRIBED;
  if (pol.n_ctas > capacity) return PL_ERR_OVERSUBSCRIBED;
  rq.pol = pol;

  pl_schedule_s* S = new (std::nothrow) pl_schedule_s();
  if (!S) return PL_ERR_OOM;
  S->comm = comm;
  S->pol = pol;
  S->timeout_ns = timeout;
  S->no_l2_hints = (flags & PL_OPT_NO_L2_HINTS) != 0;
  S->inputs_last_use = (flags & PL_OPT_INPUTS_LAST_USE) && !S->no_l2_hints;
  S->trace = (flags & PL_OPT_TRACE) != 0;
  S->overlap_launch = (flags & PL_OPT_OVERLAP_LAUNCH) != 0;
  S->stage_ahead = (flags & PL_OPT_STAGE_AHEAD) != 0;
  S->out_scale = out_scale;
  S->hook = hook;
  std::string err;
  pl_status_t st = lower(rq, &S->L, &err);
  if (st != PL_OK) {
    comm->last_error = err;
    delete S;
    return st;
  }
  // Latency regime with the grid left to the library: one queue per op a rank can run at
  // the same time, so that no ready op sits behind another in a queue.
  const bool latency = rq.n_layers == 0 && !rq.staged && S->L.message_bytes <= (1u << 20);
  if (requested == 0 && latency) {
    const int per_rank = std::min(capacity / comm->R, std::max(pol.n_ctas / comm->R, level_width(S->L, comm->R)));
    pol.n_ctas = std::max(1, per_rank) * comm->R;
    S->pol = pol;
  }
  assign_queues(&S->L, comm->R, pol.n_ctas, latency);
  if (!(flags & PL_OPT_SKIP_VALIDATE)) {
    st = validate(S->L, comm->R, &err, pol.datapath == PL_DP_TMA);
    if (st != PL_OK) {
      comm->last_error = err;
      delete S;
      return st;
    }
  }
  if (pol.datapath == PL_DP_TMA && comm->dtype != PL_U8) {
    // Plain reduce ops only (element-typed sources and destination, one destination, at most 8
    // sources): the kernel variant with the software-pipelined consumers applies.
    bool any = false, plain = true;
    for (const HostOp& op : S->L.ops) {
      if (op.kind == PL_OP_COPY) continue;
      any = true;
      if (op.bcast || op.src.size() > 8 || op.dst.dtype != comm->dtype) plain = false;
      for (const pl_ref_t& r : op.src)
        if (r.dtype != comm->dtype) plain = false;
    }
    S->pipelined_reduce = any && plain && !hook;  // the processing phase lives in the general variant
    S->pol.threads = exec_tma_threads(S->pipelined_reduce);
  }
  for (const HostOp& op : S->L.ops)
    if (op.kind == PL_OP_COPY && op.bcast) S->bcast_copies = true;
  // A window of idle SMs needs: the bulk-copy datapath with one CTA per SM, no flags (a queue
  // may be claimed late, so no queue may wait for another), one staging buffer, at most 160 SMs,
  // and ordinary launches: the claim words serve one launch at a time, and only a launch that
  // waits for everything in front of it is sure not to meet its own predecessor still running.
  if (S->pol.idle_count > 0) {
    const bool fits = pol.datapath == PL_DP_TMA && !comm->planner && S->L.n_flags == 0 && !S->stage_ahead && !S->overlap_launch &&
                      comm->sm_count <= 160 &&
                      exec_tma_max_ctas_per_sm(comm->dtype, pol.stages, pol.stage_bytes) == 1 &&
                      S->pol.n_ctas + S->pol.idle_count == comm->sm_count;
    if (!fits && idle_asked) {
      comm->last_error = "a window of idle SMs needs the bulk-copy datapath with one CTA per SM, a schedule without flags and no PL_OPT_OVERLAP_LAUNCH";
      delete S;
      return PL_ERR_UNSUPPORTED;
    }
    if (!fits) S->pol.idle_count = 0;
  }
  if (S->pol.idle_count > 0) {
    S->sm_window = true;
    for (int sm = 0; sm < comm->sm_count; ++sm)
      if (sm < S->pol.idle_first || sm >= S->pol.idle_first + S->pol.idle_count) S->sm_mask[sm >> 5] |= 1u << (sm & 31);
  }
  fill_info(S, comm->R);
  flatten(S, comm->dtype);
  if (!comm->planner) {
    st = upload(S, comm->R);
    if (st != PL_OK) {
      pl_schedule_destroy(S);
      return st;
    }
  }
  {
    std::lock_guard<std::mutex> g(comm->mu);
    comm->schedules.push_back(S);
  }
  *out = S;
  return PL_OK;
}

}  // namespace

extern "C" {
static pl_status_t check_bufs(pl_schedule_t s, const pl_bufs_t* b);
}

namespace {

void host_pipeline_destroy(pl_comm_s* comm) {
  if (comm->down_stream) cudaStreamSynchronize(static_cast<cudaStream_t>(comm->down_stream));
  if (comm->up_stream) cudaStreamSynchronize(static_cast<cudaStream_t>(comm->up_stream));
  auto drop = [](void** ev) {
    if (*ev) cudaEventDestroy(static_cast<cudaEvent_t>(*ev));
    *ev = nullptr;
  };
  drop(&comm->ev_entry);
  for (int i = 0; i < pl_comm_s::kHostSlots; ++i) {
    drop(&comm->ev_up[i]);
    drop(&comm->ev_kernel[i]);
    drop(&comm->downloads[i].done);
    comm->downloads[i].live = false;
  }
  if (comm->up_stream) cudaStreamDestroy(static_cast<cudaStream_t>(comm->up_stream));
  if (comm->down_stream) cudaStreamDestroy(static_cast<cudaStream_t>(comm->down_stream));
  comm->up_stream = comm->down_stream = nullptr;
  comm->last_download = -1;
  comm->host_calls = 0;
}

// Argument checks shared by the two host entry points.
pl_status_t check_host_bufs(pl_schedule_s* s, const pl_bufs_t* host, const pl_bufs_t* dev) {
  if (!s || !host || !dev) return PL_ERR_INVALID_ARG;
  if (s->comm->planner || !s->d_blob) return PL_ERR_UNSUPPORTED;
  pl_status_t st = check_bufs(s, dev);
  if (st != PL_OK) return st;
  for (int r = 0; r < s->comm->R; ++r) {
    if (host->in_bytes[r] < s->info.in_bytes[r] || host->out_bytes[r] < s->info.out_bytes[r]) return PL_ERR_INVALID_ARG;
    if ((s->info.in_bytes[r] && !host->in[r]) || (s->info.out_bytes[r] && !host->out[r])) return PL_ERR_INVALID_ARG;
    if (s->info.aux_bytes[r] && (!host->aux[r] || host->aux_bytes[r] < s->info.aux_bytes[r])) return PL_ERR_INVALID_ARG;
  }
  return PL_OK;
}

// host -> device copies of inputs and second operands (upload) or device -> host copies of outputs.
// skip_in: bit r set = rank r's input is already in dev->in[r] (see pl_execute_host_async).
bool copy_all(pl_schedule_s* s, int R, const pl_bufs_t* host, const pl_bufs_t* dev, bool upload, cudaStream_t on, uint32_t skip_in = 0) {
  bool ok = true;
  for (int r = 0; r < R && ok; ++r) {
    if (upload) {
      if (s->info.in_bytes[r] && !((skip_in >> r) & 1u)) {
        ok = cudaMemcpyAsync(const_cast<void*>(dev->in[r]), host->in[r], s->info.in_bytes[r], cudaMemcpyHostToDevice, on) == cudaSuccess;
        s->comm->host_h2d_bytes += s->info.in_bytes[r];
      }
      if (ok && s->info.aux_bytes[r]) {
        ok = cudaMemcpyAsync(const_cast<void*>(dev->aux[r]), host->aux[r], s->info.aux_bytes[r], cudaMemcpyHostToDevice, on) == cudaSuccess;
        s->comm->host_h2d_bytes += s->info.aux_bytes[r];
      }
    } else if (s->info.out_bytes[r]) {
      ok = cudaMemcpyAsync(host->out[r], dev->out[r], s->info.out_bytes[r], cudaMemcpyDeviceToHost, on) == cudaSuccess;
      s->comm->host_d2h_bytes += s->info.out_bytes[r];
    }
  }
  if (!ok) cudaGetLastError();
  return ok;
}

bool ranges_overlap(const std::vector<pl_comm_s::Range>& a, const std::vector<pl_comm_s::Range>& b) {
  for (const auto& x : a)
    for (const auto& y : b)
      if (x.lo < y.hi && y.lo < x.hi) return true;
  return false;
}

// Streams and events of the pipelined host entry point, created at its first use.
bool host_pipeline_init(pl_comm_s* comm) {
  if (comm->up_stream) return true;
  cudaStream_t up = nullptr, down = nullptr;
  bool ok = cudaStreamCreateWithFlags(&up, cudaStreamNonBlocking) == cudaSuccess &&
            cudaStreamCreateWithFlags(&down, cudaStreamNonBlocking) == cudaSuccess;
  auto make = [&](void** ev) {
    cudaEvent_t e = nullptr;
    ok = ok && cudaEventCreateWithFlags(&e, cudaEventDisableTiming) == cudaSuccess;
    *ev = e;
  };
  make(&comm->ev_entry);
  for (int i = 0; i < pl_comm_s::kHostSlots; ++i) {
    make(&comm->ev_up[i]);
    make(&comm->ev_kernel[i]);
    make(&comm->downloads[i].done);
  }
  comm->up_stream = up;
  comm->down_stream = down;
  if (!ok) {
    cudaGetLastError();
    host_pipeline_destroy(comm);
  }
  return ok;
}

}  // namespace

extern "C" {

const char* pl_status_string(pl_status_t st) {
  switch (st) {
    case PL_OK: return "ok";
    case PL_ERR_INVALID_ARG: return "invalid argument";
    case PL_ERR_UNSUPPORTED: return "unsupported";
    case PL_ERR_ALIGNMENT: return "misaligned pointer or size";
    case PL_ERR_OOM: return "out of memory";
    case PL_ERR_CUDA: return "CUDA error";
    case PL_ERR_TIMEOUT: return "device-side wait timed out";
    case PL_ERR_OVERSUBSCRIBED: return "more CTAs than can be co-resident";
    case PL_ERR_INVALID_SCHEDULE: return "schedule failed validation";
    case PL_ERR_OVERFLOW: return "receive capacity exceeded";
    default: return "unknown status";
  }
}

uint64_t pl_launch_count(void) { return g_launches.load(); }

static pl_status_t comm_create(int R, pl_dtype_t dtype, bool planner, pl_comm_t* out) {
  if (!out) return PL_ERR_INVALID_ARG;
  *out = nullptr;
  if (R < 2 || R > PL_MAX_RANKS) return PL_ERR_INVALID_ARG;
  if (dtype < PL_BF16 || dtype > PL_U8) return PL_ERR_INVALID_ARG;  // PL_F32X2 is internal
  pl_comm_s* c = new (std::nothrow) pl_comm_s();
  if (!c) return PL_ERR_OOM;
  c->R = R;
  c->dtype = dtype;
  c->planner = planner;
  if (!planner) {
    if (cudaGetDevice(&c->device) != cudaSuccess) { cudaGetLastError(); delete c; return PL_ERR_CUDA; }
    cudaDeviceProp prop;
    if (cudaGetDeviceProperties(&prop, c->device) != cudaSuccess) { cudaGetLastError(); delete c; return PL_ERR_CUDA; }
    c->sm_count = prop.multiProcessorCount;
    if (cudaMalloc(&c->d_status, kStatusWords * sizeof(int)) != cudaSuccess) { cudaGetLastError(); delete c; return PL_ERR_OOM; }
    if (cudaMemset(c->d_status, 0, kStatusWords * sizeof(int)) != cudaSuccess) { cudaGetLastError(); cudaFree(c->d_status); delete c; return PL_ERR_CUDA; }
    cudaStream_t st = nullptr;
    if (cudaStreamCreateWithFlags(&st, cudaStreamNonBlocking) != cudaSuccess) { cudaGetLastError(); cudaFree(c->d_status); delete c; return PL_ERR_CUDA; }
    c->status_stream = st;
  }
  *out = c;
  return PL_OK;
}

pl_status_t pl_comm_create(int R, pl_dtype_t dtype, pl_comm_t* out) { return comm_create(R, dtype, false, out); }
pl_status_t pl_comm_create_planner(int R, pl_dtype_t dtype, pl_comm_t* out) { return comm_create(R, dtype, true, out); }

pl_status_t pl_comm_destroy(pl_comm_t comm) {
  if (!comm) return PL_ERR_INVALID_ARG;
  if (!comm->schedules.empty() || comm->n_plans != 0) return PL_ERR_INVALID_ARG;
  if (comm->d_status) cudaFree(comm->d_status);
  if (comm->status_stream) cudaStreamDestroy(static_cast<cudaStream_t>(comm->status_stream));
  host_pipeline_destroy(comm);
  delete comm;
  return PL_OK;
}

pl_status_t pl_comm_tune(pl_comm_t comm, void* stream, int32_t* push_ctas_out, int32_t* idle_sm_first_out, int32_t* idle_sm_count_out) {
  if (!comm) return PL_ERR_INVALID_ARG;
  if (push_ctas_out) *push_ctas_out = 0;
  if (idle_sm_first_out) *idle_sm_first_out = 0;
  if (idle_sm_count_out) *idle_sm_count_out = 0;
  if (comm->planner) return PL_ERR_UNSUPPORTED;
  if (!on_comm_device(comm)) return PL_ERR_INVALID_ARG;
  const int R = comm->R;
  const size_t es = (size_t)elem_size(comm->dtype);
  // the measured case: an all-gather of 64 MiB (R contributions of 64 MiB / R), far beyond L2
  const size_t part = ((size_t)64 << 20) / (size_t)R / (16 * es) * (16 * es);
  const size_t count = part / es;
  // The all-gather is measured where it usually runs: behind the reduce-scatter that produces its
  // input (both with their inputs marked last-use), so that it finds that input in L2 and its
  // DRAM traffic is almost purely writes.  Alone, with its input coming from DRAM, another
  // candidate can be the fastest (on one B200: 136 CTAs alone, 128 CTAs behind a reduce-scatter).
  char *d_src = nullptr, *d_in = nullptr, *d_out = nullptr;
  if (cudaMalloc(&d_src, part * R * R) != cudaSuccess || cudaMalloc(&d_in, part * R) != cudaSuccess ||
      cudaMalloc(&d_out, part * R * R) != cudaSuccess) {
    cudaGetLastError();
    if (d_src) cudaFree(d_src);
    if (d_in) cudaFree(d_in);
    return PL_ERR_OOM;
  }
  cudaStream_t cs = static_cast<cudaStream_t>(stream);
  cudaMemsetAsync(d_src, 0, part * R * R, cs);
  cudaMemsetAsync(d_in, 0, part * R, cs);
  cudaEvent_t e0 = nullptr, e1 = nullptr;
  cudaEventCreate(&e0);
  cudaEventCreate(&e1);
  pl_bufs_t bufs;
  std::memset(&bufs, 0, sizeof(bufs));
  pl_bufs_t rs_bufs;
  std::memset(&rs_bufs, 0, sizeof(rs_bufs));
  for (int r = 0; r < R; ++r) {
    bufs.in[r] = d_in + (size_t)r * part;
    bufs.in_bytes[r] = part;
    bufs.out[r] = d_out + (size_t)r * part * R;
    bufs.out_bytes[r] = part * R;
    rs_bufs.in[r] = d_src + (size_t)r * part * R;
    rs_bufs.in_bytes[r] = part * R;
    rs_bufs.out[r] = d_in + (size_t)r * part;
    rs_bufs.out_bytes[r] = part;
  }
  pl_schedule_t rs = nullptr;
  {
    pl_sched_opts_t o;
    std::memset(&o, 0, sizeof(o));
    o.struct_size = sizeof(o);
    o.datapath = PL_DP_TMA;
    o.flags = PL_OPT_INPUTS_LAST_USE;
    if (pl_schedule_build(comm, PL_REDUCE_SCATTER, PL_ALGO_DIRECT, count * R, (size_t)1 << 20, &o, &rs) != PL_OK) rs = nullptr;
  }
  const int per_sm = exec_tma_max_ctas_per_sm(comm->dtype, 4, 48 * 1024);
  const int resident = std::max(1, per_sm) * comm->sm_count;
  // candidates: plain launches of every multiple of R down to 3/4 of the resident CTAs, and, with
  // one CTA per SM, the same grids with the idle SMs as a window at a few places of the SM range
  struct Cand { int n_ctas, idle_first, idle_count; };
  std::vector<Cand> cands;
  const int firsts[] = {0, 8, 16, 64};
  for (int g = resident / R * R; g >= resident * 3 / 4 && g >= R; g -= R) {
    cands.push_back({g, 0, 0});
    const int idle = comm->sm_count - g;
    if (per_sm == 1 && comm->sm_count <= 160 && idle >= 12 && idle <= 40)
      for (int f : firsts)
        if (f + idle <= comm->sm_count) cands.push_back({g, f, idle});
  }
  Cand best{0, 0, 0};
  float best_ms = 0.f;
  pl_status_t result = PL_OK;
  const Cand saved{comm->tuned_push_ctas, comm->tuned_idle_first, comm->tuned_idle_count};
  for (const Cand& cd : cands) {
    pl_sched_opts_t o;
    std::memset(&o, 0, sizeof(o));
    o.struct_size = sizeof(o);
    o.n_ctas = cd.n_ctas;
    o.datapath = PL_DP_TMA;
    o.flags = PL_OPT_INPUTS_LAST_USE;
    o.idle_sm_first = cd.idle_first;
    o.idle_sm_count = cd.idle_count;
    pl_schedule_t s = nullptr;
    if (pl_schedule_build(comm, PL_ALLGATHER, PL_ALGO_DIRECT, count, (size_t)1 << 20, &o, &s) != PL_OK) continue;
    bool ok = true;
    auto pair = [&]() { return (!rs || pl_execute(rs, &rs_bufs, stream) == PL_OK) && pl_execute(s, &bufs, stream) == PL_OK; };
    for (int i = 0; i < 2 && ok; ++i) ok = pair();
    const int reps = 10;
    ok = ok && cudaEventRecord(e0, cs) == cudaSuccess;
    for (int i = 0; i < reps && ok; ++i) ok = pair();
    ok = ok && cudaEventRecord(e1, cs) == cudaSuccess && cudaEventSynchronize(e1) == cudaSuccess;
    float ms = 0.f;
    ok = ok && cudaEventElapsedTime(&ms, e0, e1) == cudaSuccess;
    pl_schedule_destroy(s);
    if (!ok) {
      cudaGetLastError();
      result = PL_ERR_CUDA;
      break;
    }
    // Candidates run from the largest grid down, plain launch first: a later one replaces the
    // pick only if it is faster by more than the noise of the measurement (0.5 %), so that equal
    // candidates resolve to the larger grid and to the plain launch.
    if (best.n_ctas == 0 || ms < best_ms * 0.995f) {
      best = cd;
      best_ms = ms;
    }
  }
  cudaStreamSynchronize(cs);
  cudaEventDestroy(e0);
  cudaEventDestroy(e1);
  if (rs) pl_schedule_destroy(rs);
  cudaFree(d_src);
  cudaFree(d_in);
  cudaFree(d_out);
  const Cand pick = (result == PL_OK && best.n_ctas > 0) ? best : saved;
  comm->tuned_push_ctas = pick.n_ctas;
  comm->tuned_idle_first = pick.idle_first;
  comm->tuned_idle_count = pick.idle_count;
  if (push_ctas_out) *push_ctas_out = pick.n_ctas;
  if (idle_sm_first_out) *idle_sm_first_out = pick.idle_first;
  if (idle_sm_count_out) *idle_sm_count_out = pick.idle_count;
  return result;
}

pl_status_t pl_comm_status(pl_comm_t comm, pl_devstatus_t* out) {
  if (!comm || !out) return PL_ERR_INVALID_ARG;
  std::memset(out, 0, sizeof(*out));
  if (comm->planner) return PL_OK;
  if (!on_comm_device(comm)) return PL_ERR_INVALID_ARG;
  int words[kStatusWords];
  // the record as it stands now, read on a stream of its own: no other stream is waited for
  cudaStream_t st = static_cast<cudaStream_t>(comm->status_stream);
  if (cudaMemcpyAsync(words, comm->d_status, sizeof(words), cudaMemcpyDeviceToHost, st) != cudaSuccess ||
      cudaStreamSynchronize(st) != cudaSuccess) {
    cudaGetLastError();
    return PL_ERR_CUDA;
  }
  out->code = words[0];
  out->queue = words[1];
  out->op = words[2];
  out->flag = words[3];
  std::memcpy(&out->expected, words + 4, 8);
  std::memcpy(&out->observed, words + 6, 8);
  return PL_OK;
}

const char* pl_comm_last_error(pl_comm_t comm) { return comm ? comm->last_error.c_str() : ""; }

pl_status_t pl_comm_reset(pl_comm_t comm, void* stream) {
  if (!comm) return PL_ERR_INVALID_ARG;
  if (comm->planner) return PL_OK;
  if (!on_comm_device(comm)) return PL_ERR_INVALID_ARG;
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  if (cudaMemsetAsync(comm->d_status, 0, kStatusWords * sizeof(int), st) != cudaSuccess) { cudaGetLastError(); return PL_ERR_CUDA; }
  std::lock_guard<std::mutex> g(comm->mu);
  for (pl_schedule_s* S : comm->schedules) {
    if (S->d_blob && cudaMemsetAsync(S->d_blob + S->off_flags, 0, S->sync_bytes, st) != cudaSuccess) { cudaGetLastError(); return PL_ERR_CUDA; }
    // packet tags restart with the epoch: old packets must not match them
    if (S->packet_ctas_per_rank && S->d_scratch && cudaMemsetAsync(S->d_scratch, 0, S->scratch_total, st) != cudaSuccess) { cudaGetLastError(); return PL_ERR_CUDA; }
  }
  return PL_OK;
}

pl_status_t pl_schedule_build(pl_comm_t comm, pl_collective_t coll, pl_algo_t algo, size_t count_per_rank,
                              size_t chunk_bytes, const pl_sched_opts_t* opts, pl_schedule_t* out) {
  if (coll < PL_ALLREDUCE || coll > PL_ALLTOALL) return PL_ERR_INVALID_ARG;  // V and rooted forms have their own calls
  BuildRequest rq{};
  rq.coll = coll;
  rq.algo = algo;
  if (algo == PL_ALGO_AUTO && comm) {
    const size_t bytes = count_per_rank * (size_t)elem_size(comm->dtype);
    rq.algo = coll != PL_ALLREDUCE ? PL_ALGO_DIRECT : bytes <= (32u << 10) ? PL_ALGO_ONESHOT : PL_ALGO_DIRECT_FUSED;
  }
  rq.count_per_rank = count_per_rank;
  rq.chunk_bytes = chunk_bytes;
  return build_common(comm, rq, opts, out);
}

pl_status_t pl_schedule_build_v(pl_comm_t comm, pl_collective_t coll, pl_algo_t algo, const size_t* counts,
                                size_t chunk_bytes, const pl_sched_opts_t* opts, pl_schedule_t* out) {
  if (!comm || !counts) return PL_ERR_INVALID_ARG;
  if (coll != PL_ALLTOALLV && coll != PL_ALLGATHERV && coll != PL_REDUCE_SCATTERV) return PL_ERR_UNSUPPORTED;
  std::vector<uint64_t> c(coll == PL_ALLTOALLV ? (size_t)comm->R * comm->R : (size_t)comm->R);
  for (size_t i = 0; i < c.size(); ++i) c[i] = counts[i];
  BuildRequest rq{};
  rq.coll = coll;
  rq.algo = algo == PL_ALGO_AUTO ? PL_ALGO_DIRECT : algo;
  rq.chunk_bytes = chunk_bytes;
  rq.counts_v = c.data();
  return build_common(comm, rq, opts, out);
}

pl_status_t pl_schedule_build_rooted(pl_comm_t comm, pl_collective_t coll, int root, size_t count_per_rank,
                                     size_t chunk_bytes, const pl_sched_opts_t* opts, pl_schedule_t* out) {
  if (!comm) return PL_ERR_INVALID_ARG;
  if (coll != PL_BROADCAST && coll != PL_REDUCE && coll != PL_SCATTER && coll != PL_GATHER) return PL_ERR_INVALID_ARG;
  if (root < 0 || root >= comm->R) return PL_ERR_INVALID_ARG;
  BuildRequest rq{};
  rq.coll = coll;
  rq.algo = PL_ALGO_DIRECT;
  rq.root = root;
  rq.count_per_rank = count_per_rank;
  rq.chunk_bytes = chunk_bytes;
  return build_common(comm, rq, opts, out);
}

pl_status_t pl_schedule_build_layers(pl_comm_t comm, pl_algo_t algo, size_t count_per_rank, int n_layers,
                                     const pl_sched_opts_t* opts, pl_schedule_t* out) {
  if (n_layers < 1) return PL_ERR_INVALID_ARG;
  BuildRequest rq{};
  rq.coll = PL_ALLREDUCE;
  rq.algo = algo == PL_ALGO_AUTO ? PL_ALGO_DIRECT_FUSED : algo;  // the fastest layered form at 16 KiB - 1 MiB
  if (algo == PL_ALGO_AUTO && opts && opts->struct_size == sizeof(pl_sched_opts_t) && opts->datapath == PL_DP_PACKET) rq.algo = PL_ALGO_ONESHOT;
  // Everything left to the library and a message of at most 4 KiB: the packet datapath with one
  // CTA per rank is the fastest layered form there (1.8-2.05 us per layer against 2.0-2.2 us with flags).
  pl_sched_opts_t packet_opts;
  if (algo == PL_ALGO_AUTO && comm && comm->dtype != PL_U8 && count_per_rank * (size_t)elem_size(comm->dtype) <= 4096 &&
      (count_per_rank * (size_t)elem_size(comm->dtype)) % 16 == 0 &&
      (!opts || (opts->struct_size == sizeof(pl_sched_opts_t) && opts->datapath == PL_DP_AUTO && opts->n_ctas == 0 && opts->threads == 0 &&
                 opts->hook == 0 && !(opts->flags & PL_OPT_STAGED)))) {
    std::memset(&packet_opts, 0, sizeof(packet_opts));
    if (opts) packet_opts = *opts;
    packet_opts.struct_size = sizeof(pl_sched_opts_t);
    packet_opts.datapath = PL_DP_PACKET;
    rq.algo = PL_ALGO_ONESHOT;
    opts = &packet_opts;
  }
  rq.count_per_rank = count_per_rank;
  rq.n_layers = n_layers;
  // a layer is one chunk per partition: the latency path does not pipeline inside a layer
  rq.chunk_bytes = ((uint64_t)1 << 40);
  return build_common(comm, rq, opts, out);
}

pl_status_t pl_schedule_info(pl_schedule_t s, pl_sched_info_t* out) {
  if (!s || !out) return PL_ERR_INVALID_ARG;
  *out = s->info;
  return PL_OK;
}

pl_status_t pl_schedule_dump(pl_schedule_t s, pl_op_t* ops, size_t cap, size_t* n) {
  if (!s || !n) return PL_ERR_INVALID_ARG;
  *n = s->L.ops.size();
  if (!ops) return PL_OK;
  const size_t m = std::min(cap, s->L.ops.size());
  for (size_t i = 0; i < m; ++i) {
    const HostOp& h = s->L.ops[i];
    pl_op_t& o = ops[i];
    std::memset(&o, 0, sizeof(o));
    o.kind = h.kind;
    o.exec_rank = h.exec_rank;
    o.queue = h.queue;
    o.topo = h.topo;
    o.layer = h.layer;
    o.n_src = (int32_t)h.src.size();
    o.n_wait = (int32_t)h.waits.size();
    o.signal_flag = h.signal;
    o.signal_flag2 = h.signal2;
    o.dst_bcast = (h.bcast ? 1 : 0) | (h.final_hook ? 2 : 0) | (h.stage_ahead ? 4 : 0);
    o.count = h.count;
    o.dst = h.dst;
    for (size_t k = 0; k < h.src.size(); ++k) o.src[k] = h.src[k];
    for (size_t k = 0; k < h.waits.size(); ++k) {
      o.wait_flag[k] = h.waits[k];
      o.wait_need[k] = s->L.flag_need[h.waits[k]];
    }
  }
  return PL_OK;
}

pl_status_t pl_schedule_validate(pl_schedule_t s, char* msg, size_t msg_cap) {
  if (!s) return PL_ERR_INVALID_ARG;
  std::string err;
  pl_status_t st = validate(s->L, s->comm->R, &err, s->pol.datapath == PL_DP_TMA);
  if (msg && msg_cap) {
    std::snprintf(msg, msg_cap, "%s", err.c_str());
  }
  return st;
}

pl_status_t pl_schedule_trace_read(pl_schedule_t s, uint64_t* out, size_t cap_entries, void* stream) {
  if (!s || !out || !s->trace || !s->d_blob) return PL_ERR_INVALID_ARG;
  if (cap_entries < 2 * s->L.ops.size()) return PL_ERR_INVALID_ARG;
  if (cudaStreamSynchronize(static_cast<cudaStream_t>(stream)) != cudaSuccess ||
      cudaMemcpy(out, s->d_blob + s->off_trace, 2 * s->L.ops.size() * sizeof(unsigned long long), cudaMemcpyDeviceToHost) != cudaSuccess) {
    cudaGetLastError();
    return PL_ERR_CUDA;
  }
  return PL_OK;
}

pl_status_t pl_schedule_debug_drop_wait(pl_schedule_t s, size_t op_index) {
  if (!s || op_index >= s->L.ops.size()) return PL_ERR_INVALID_ARG;
  HostOp& h = s->L.ops[op_index];
  if (h.waits.empty()) return PL_ERR_INVALID_ARG;
  h.waits.erase(h.waits.begin());
  return PL_OK;
}

pl_status_t pl_schedule_debug_break_wait(pl_schedule_t s, size_t op_index) {
  if (!s || op_index >= s->L.ops.size()) return PL_ERR_INVALID_ARG;
  const HostOp& h = s->L.ops[op_index];
  if (h.waits.empty()) return PL_ERR_INVALID_ARG;
  if (s->packet_ctas_per_rank) {  // no wait entries on the device: the op's polls expect a tag nobody publishes
    s->packet_break_op = (long long)op_index;
    return PL_OK;
  }
  const size_t pos = (size_t)s->topo_to_dev[op_index];
  DevWait& w = s->waits[pos * s->wait_stride];
  w.need += 1;  // one more signal than the schedule will ever produce
  if (s->d_blob) {
    if (cudaMemcpy(s->d_blob + s->off_waits + (pos * s->wait_stride) * sizeof(DevWait), &w, sizeof(DevWait),
                   cudaMemcpyHostToDevice) != cudaSuccess) {
      cudaGetLastError();
      return PL_ERR_CUDA;
    }
  }
  return PL_OK;
}

pl_status_t pl_schedule_destroy(pl_schedule_t s) {
  if (!s) return PL_ERR_INVALID_ARG;
  if (s->d_blob) cudaFree(s->d_blob);
  if (s->d_scratch) cudaFree(s->d_scratch);
  if (s->comm) {
    std::lock_guard<std::mutex> g(s->comm->mu);
    auto& v = s->comm->schedules;
    for (size_t i = 0; i < v.size(); ++i)
      if (v[i] == s) { v.erase(v.begin() + i); break; }
  }
  delete s;
  return PL_OK;
}

static pl_status_t check_bufs(pl_schedule_t s, const pl_bufs_t* b) {
  const int R = s->comm->R;
  for (int r = 0; r < R; ++r) {
    const bool need_in = s->info.in_bytes[r] > 0, need_out = s->info.out_bytes[r] > 0;
    if ((need_in && !b->in[r]) || (need_out && !b->out[r])) return PL_ERR_INVALID_ARG;
    if (((uintptr_t)b->in[r] & 15) || ((uintptr_t)b->out[r] & 15)) return PL_ERR_ALIGNMENT;
    if (b->in_bytes[r] < s->info.in_bytes[r] || b->out_bytes[r] < s->info.out_bytes[r]) return PL_ERR_INVALID_ARG;
  }
  for (int r = 0; r < R; ++r) {
    if (!s->info.aux_bytes[r]) continue;
    if (!b->aux[r] || b->aux_bytes[r] < s->info.aux_bytes[r]) return PL_ERR_INVALID_ARG;
    if ((uintptr_t)b->aux[r] & 15) return PL_ERR_ALIGNMENT;
  }
  // outputs must not overlap any input or another output (all collectives are out of place)
  for (int r = 0; r < R; ++r) {
    const uintptr_t olo = (uintptr_t)b->out[r], ohi = olo + s->info.out_bytes[r];
    if (olo == ohi) continue;
    for (int p = 0; p < R; ++p) {
      const uintptr_t ilo = (uintptr_t)b->in[p], ihi = ilo + s->info.in_bytes[p];
      if (ilo < ohi && olo < ihi) return PL_ERR_INVALID_ARG;
      const uintptr_t alo = (uintptr_t)b->aux[p], ahi = alo + s->info.aux_bytes[p];
      if (s->info.aux_bytes[p] && alo < ohi && olo < ahi) return PL_ERR_INVALID_ARG;
      if (p != r) {
        const uintptr_t qlo = (uintptr_t)b->out[p], qhi = qlo + s->info.out_bytes[p];
        if (qlo < ohi && olo < qhi) return PL_ERR_INVALID_ARG;
      }
    }
  }
  return PL_OK;
}

pl_status_t pl_execute(pl_schedule_t s, const pl_bufs_t* bufs, void* stream) {
  if (!s || !bufs) return PL_ERR_INVALID_ARG;
  if (s->comm->planner || !s->d_blob) return PL_ERR_UNSUPPORTED;
  if (!on_comm_device(s->comm)) return PL_ERR_INVALID_ARG;
  pl_status_t st = check_bufs(s, bufs);
  if (st != PL_OK) return st;
  if (s->packet_ctas_per_rank) {
    PacketParams K;
    std::memset(&K, 0, sizeof(K));
    const int R = s->comm->R;
    for (int r = 0; r < R; ++r) {
      K.in[r] = bufs->in[r];
      K.out[r] = bufs->out[r];
      K.pkt[r] = s->d_scratch + s->scratch_off[r];
    }
    K.epoch = reinterpret_cast<unsigned long long*>(s->d_blob + s->off_epoch);
    K.status = s->comm->d_status;
    K.trace = s->trace ? reinterpret_cast<unsigned long long*>(s->d_blob + s->off_trace) : nullptr;
    K.timeout_ns = s->timeout_ns;
    K.units_per_rank = s->L.message_bytes / 16;
    K.n_ranks = R;
    K.n_layers = s->L.n_layers;
    K.ctas_per_rank = s->packet_ctas_per_rank;
    K.out_scale = s->out_scale;
    K.break_op = s->packet_break_op;
    if (launch_exec_packet(s->comm->dtype, K, s->pol.threads, s->overlap_launch, static_cast<cudaStream_t>(stream)) != cudaSuccess) {
      cudaGetLastError();
      return PL_ERR_CUDA;
    }
    g_launches.fetch_add(1);
    return PL_OK;
  }
  ExecParams P;
  std::memset(&P, 0, sizeof(P));
  const int R = s->comm->R;
  for (int r = 0; r < R; ++r) {
    P.base[kSlotIn + r] = const_cast<void*>(bufs->in[r]);
    P.base[kSlotOut + r] = bufs->out[r];
    P.base[kSlotScratch + r] = s->d_scratch ? s->d_scratch + s->scratch_off[r] : nullptr;
    P.base[kSlotAux + r] = s->info.aux_bytes[r] ? const_cast<void*>(bufs->aux[r]) : nullptr;
  }
  P.hook = s->hook;
  P.stage_ahead = s->stage_ahead ? 1u : 0u;
  P.n_flags = (uint32_t)s->L.n_flags;
  P.scratch_half = s->scratch_half;
  P.ops = reinterpret_cast<const DevOp*>(s->d_blob + s->off_ops);
  P.n_queues = (uint32_t)s->pol.n_ctas;
  P.srcs = reinterpret_cast<const uint64_t*>(s->d_blob + s->off_srcs);
  P.waits = reinterpret_cast<const DevWait*>(s->d_blob + s->off_waits);
  P.src_stride = s->src_stride;
  P.wait_stride = s->wait_stride;
  P.flags = s->L.n_flags ? reinterpret_cast<unsigned long long*>(s->d_blob + s->off_flags) : nullptr;
  P.epoch = reinterpret_cast<unsigned long long*>(s->d_blob + s->off_epoch);
  P.status = s->comm->d_status;
  P.trace = s->trace ? reinterpret_cast<unsigned long long*>(s->d_blob + s->off_trace) : nullptr;
  P.sm_state = s->sm_window ? reinterpret_cast<unsigned long long*>(s->d_blob + s->off_sm_state) : nullptr;
  for (int i = 0; i < 5; ++i) P.sm_mask[i] = s->sm_mask[i];
  P.timeout_ns = s->timeout_ns;
  P.n_ranks = R;
  P.stages = s->pol.stages;
  P.stage_bytes = s->pol.stage_bytes;
  // bulk stores stream out (evict-first), sources of copies are re-read by other ranks (evict-last)
  P.hints = s->no_l2_hints ? 0u : (6u | (s->inputs_last_use ? 1u : 0u));
  P.out_scale = s->out_scale;
  P.overlap_launch = s->overlap_launch ? 1u : 0u;
  P.pipelined_reduce = s->pipelined_reduce ? 1u : 0u;
  P.bcast_copies = s->bcast_copies ? 1u : 0u;
  cudaError_t le = s->pol.datapath == PL_DP_TMA
                       ? launch_exec_tma(s->comm->dtype, P, s->sm_window ? s->comm->sm_count : s->pol.n_ctas, static_cast<cudaStream_t>(stream))
                       : launch_exec(s->comm->dtype, P, s->pol.n_ctas, s->pol.threads, static_cast<cudaStream_t>(stream));
  if (le != cudaSuccess) return PL_ERR_CUDA;
  g_launches.fetch_add(1);
  return PL_OK;
}

pl_status_t pl_execute_host(pl_schedule_t s, const pl_bufs_t* host, const pl_bufs_t* dev, void* stream) {
  pl_status_t st = check_host_bufs(s, host, dev);
  if (st != PL_OK) return st;
  const int R = s->comm->R;
  cudaStream_t cs = static_cast<cudaStream_t>(stream);
  // downloads of earlier pipelined host executes may still read or write what this call touches
  st = pl_comm_host_fence(s->comm, stream);
  if (st != PL_OK) return st;
  if (!copy_all(s, R, host, dev, /*upload=*/true, cs)) return PL_ERR_CUDA;
  st = pl_execute(s, dev, stream);
  if (st != PL_OK) return st;
  if (!copy_all(s, R, host, dev, /*upload=*/false, cs)) return PL_ERR_CUDA;
  return PL_OK;
}

pl_status_t pl_execute_host_async(pl_schedule_t s, const pl_bufs_t* host, const pl_bufs_t* dev, void* stream) {
  pl_status_t st = check_host_bufs(s, host, dev);
  if (st != PL_OK) return st;
  pl_comm_s* comm = s->comm;
  if (!on_comm_device(comm)) return PL_ERR_INVALID_ARG;
  std::lock_guard<std::mutex> host_guard(comm->host_mu);
  if (!host_pipeline_init(comm)) return PL_ERR_CUDA;
  const int R = comm->R;
  cudaStream_t cs = static_cast<cudaStream_t>(stream);
  cudaStream_t up = static_cast<cudaStream_t>(comm->up_stream), down = static_cast<cudaStream_t>(comm->down_stream);
  const int slot = (int)(comm->host_calls % pl_comm_s::kHostSlots);
  bool ok = true;
  auto wait = [&](cudaStream_t on, void* ev) { ok = ok && cudaStreamWaitEvent(on, static_cast<cudaEvent_t>(ev), 0) == cudaSuccess; };

  // The slot's events are about to be recorded again: whoever still waits for the download that
  // used it kHostSlots calls ago must have seen it first.
  pl_comm_s::Download& mine = comm->downloads[slot];
  if (mine.live) {
    wait(up, mine.done);
    wait(cs, mine.done);
    mine.live = false;
  }
  // Uploads overwrite the device inputs: the schedule of the previous host execute (and, on a
  // stream in order, everything before it) must have finished reading them.  The first call, or a
  // change of stream, also orders them behind what the caller has put on `stream` so far.
  if (comm->host_calls == 0 || comm->host_stream_last != stream) {
    ok = ok && cudaEventRecord(static_cast<cudaEvent_t>(comm->ev_entry), cs) == cudaSuccess;
    wait(up, comm->ev_entry);
  }
  if (comm->host_calls > 0) wait(up, comm->ev_kernel[(comm->host_calls - 1) % pl_comm_s::kHostSlots]);
  // Hazards with downloads still in flight: an upload must not read a host range, nor overwrite a
  // device range, that a download has yet to finish with; the schedule must not overwrite device
  // outputs that a download still reads.
  // Forwarding: an input whose host buffer is exactly what the previous call's download is still
  // writing, and whose device buffer is exactly what that download reads, is already where the
  // upload would put it (the previous schedule wrote it there): no upload, and nothing to wait
  // for (a reduce-scatter's result handed to an all-gather through a host buffer).  Only the
  // immediately preceding call is looked at, and only while its download is in flight: once it
  // has completed the caller may have rewritten the host buffer.
  uint32_t fwd = 0;
  if (comm->last_download >= 0 && comm->host_stream_last == stream) {  // same stream: the previous schedule is ordered in front of this one
    pl_comm_s::Download& d = comm->downloads[comm->last_download];
    if (d.live && cudaEventQuery(static_cast<cudaEvent_t>(d.done)) != cudaSuccess && d.host_out.size() == d.dev_out.size()) {
      for (int r = 0; r < R; ++r) {
        const size_t n = s->info.in_bytes[r];
        if (!n) continue;
        for (size_t k = 0; k < d.host_out.size(); ++k)
          if (d.host_out[k].lo == static_cast<const char*>(host->in[r]) && (size_t)(d.host_out[k].hi - d.host_out[k].lo) == n &&
              d.dev_out[k].lo == static_cast<const char*>(dev->in[r]) && (size_t)(d.dev_out[k].hi - d.dev_out[k].lo) == n)
            fwd |= 1u << r;
      }
    }
    cudaGetLastError();  // cudaErrorNotReady is not an error here
  }
  std::vector<pl_comm_s::Range> h_in, d_in, d_out, h_out;
  for (int r = 0; r < R; ++r) {
    auto add = [](std::vector<pl_comm_s::Range>& v, const void* p, size_t n) {
      if (p && n) v.push_back({static_cast<const char*>(p), static_cast<const char*>(p) + n});
    };
    if (!((fwd >> r) & 1u)) {
      add(h_in, host->in[r], s->info.in_bytes[r]);
      add(d_in, dev->in[r], s->info.in_bytes[r]);
    }
    add(h_in, host->aux[r], s->info.aux_bytes[r]);
    add(d_in, dev->aux[r], s->info.aux_bytes[r]);
    add(d_out, dev->out[r], s->info.out_bytes[r]);
    add(h_out, host->out[r], s->info.out_bytes[r]);
  }
  for (pl_comm_s::Download& d : comm->downloads) {
    if (!d.live) continue;
    if (cudaEventQuery(static_cast<cudaEvent_t>(d.done)) == cudaSuccess) {
      d.live = false;
      continue;
    }
    cudaGetLastError();  // cudaErrorNotReady is not an error here
    if (ranges_overlap(h_in, d.host_out) || ranges_overlap(d_in, d.dev_out)) wait(up, d.done);
    if (ranges_overlap(d_out, d.dev_out) || ranges_overlap(d_in, d.dev_out)) wait(cs, d.done);
  }
  if (!ok) { cudaGetLastError(); return PL_ERR_CUDA; }

  if (!copy_all(s, R, host, dev, /*upload=*/true, up, fwd)) return PL_ERR_CUDA;
  ok = cudaEventRecord(static_cast<cudaEvent_t>(comm->ev_up[slot]), up) == cudaSuccess;
  wait(cs, comm->ev_up[slot]);
  if (!ok) { cudaGetLastError(); return PL_ERR_CUDA; }
  st = pl_execute(s, dev, stream);
  if (st != PL_OK) return st;
  ok = cudaEventRecord(static_cast<cudaEvent_t>(comm->ev_kernel[slot]), cs) == cudaSuccess;
  wait(down, comm->ev_kernel[slot]);
  if (!ok) { cudaGetLastError(); return PL_ERR_CUDA; }
  ++comm->host_calls;                 // ev_kernel[slot] is what the next upload waits for
  comm->host_stream_last = stream;
  if (!copy_all(s, R, host, dev, /*upload=*/false, down)) return PL_ERR_CUDA;
  if (cudaEventRecord(static_cast<cudaEvent_t>(mine.done), down) != cudaSuccess) { cudaGetLastError(); return PL_ERR_CUDA; }
  mine.host_out = std::move(h_out);
  mine.dev_out = std::move(d_out);
  mine.live = true;
  comm->last_download = slot;
  return PL_OK;
}

pl_status_t pl_comm_host_stats(pl_comm_t comm, uint64_t* h2d_bytes, uint64_t* d2h_bytes) {
  if (!comm) return PL_ERR_INVALID_ARG;
  std::lock_guard<std::mutex> host_guard(comm->host_mu);
  if (h2d_bytes) *h2d_bytes = comm->host_h2d_bytes;
  if (d2h_bytes) *d2h_bytes = comm->host_d2h_bytes;
  return PL_OK;
}

pl_status_t pl_comm_host_fence(pl_comm_t comm, void* stream) {
  if (!comm) return PL_ERR_INVALID_ARG;
  std::lock_guard<std::mutex> host_guard(comm->host_mu);
  if (comm->last_download < 0) return PL_OK;
  // downloads run in order on one stream: the last one's event covers them all
  if (cudaStreamWaitEvent(static_cast<cudaStream_t>(stream), static_cast<cudaEvent_t>(comm->downloads[comm->last_download].done), 0) != cudaSuccess) {
    cudaGetLastError();
    return PL_ERR_CUDA;
  }
  return PL_OK;
}

pl_status_t pl_comm_host_sync(pl_comm_t comm) {
  if (!comm) return PL_ERR_INVALID_ARG;
  std::lock_guard<std::mutex> host_guard(comm->host_mu);
  if (comm->last_download < 0) return PL_OK;
  if (cudaEventSynchronize(static_cast<cudaEvent_t>(comm->downloads[comm->last_download].done)) != cudaSuccess) {
    cudaGetLastError();
    return PL_ERR_CUDA;
  }
  for (pl_comm_s::Download& d : comm->downloads) d.live = false;
  return PL_OK;
}

}  // extern "C"
