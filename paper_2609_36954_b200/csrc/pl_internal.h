// Internal types shared by the host orchestrator, the C-ABI layer and the kernels.
#pragma once
#include <cstdint>
#include <string>
#include <utility>
#include <vector>

#include "purlin.h"

namespace pl {

inline int elem_size(int dtype) {
  switch (dtype) {
    case PL_BF16: return 2;
    case PL_F32: return 4;
    case PL_I32: return 4;
    case PL_F32X2: return 8;
    default: return 1;
  }
}
// Element type of partial sums that travel between ops (ring hops, tree levels).
// bf16 data: fp32.  fp32 data: a compensated (sum, correction) fp32 pair, so that rounding once
// per hop does not eat the fp32 tolerance.  int32: int32.
inline int partial_dtype(int dtype) { return dtype == PL_BF16 ? PL_F32 : dtype == PL_F32 ? PL_F32X2 : dtype; }

struct HostOp {
  int kind = PL_OP_COPY;
  int exec_rank = 0;
  int layer = 0;
  uint64_t count = 0;  // elements (bytes for COPY)
  pl_ref_t dst{};
  bool bcast = false;
  std::vector<pl_ref_t> src;
  std::vector<int> waits;  // flag ids
  int signal = -1;
  int signal2 = -1;
  bool stage_ahead = false;  // a stage op that waits for nothing (double-buffered staging may run it early)
  bool final_hook = false;  // writes final output: the processing phase (residual, fp32 output) applies
  int role = 0;  // 0 = any queue of the rank; 1 stage, 2 reduce, 3 gather: CTA groups per role (Sec. 3.2)
  int queue = -1;
  int topo = -1;
};

// ---- device-resident schedule ------------------------------------------------------
// A buffer address is packed as (slot << 48) | byte offset; slot indexes the pointer
// table passed by value in the kernel parameters: in[0..16), out[16..32), scratch[32..48).
constexpr int kSlotIn = 0, kSlotOut = PL_MAX_RANKS, kSlotScratch = 2 * PL_MAX_RANKS, kSlotAux = 3 * PL_MAX_RANKS;
constexpr int kNumSlots = 4 * PL_MAX_RANKS;
constexpr uint32_t kNoFlag = 0xFFFFFFFFu;
constexpr uint32_t kNopKind = 0xFFu;  // placeholder op of an empty queue

struct alignas(16) DevOp {
  uint32_t kind;        // pl_op_kind_t
  uint32_t n_src;
  uint32_t remaining;   // ops that follow this one in its queue
  uint32_t src_f32_mask;  // bit p set: source p holds partials (fp32 for bf16 data, fp32 pairs for fp32 data)
  uint32_t rsv1;
  uint32_t n_wait;
  uint32_t signal;      // flag index or kNoFlag
  uint32_t flags;       // bit0: dst holds partials (or fp32 output); bit1: dst broadcast; bit2: final op of a hooked schedule
  uint64_t count;       // elements (bytes for COPY)
  uint64_t dst;         // packed address
  uint32_t topo;
  uint32_t signal2;     // second flag index or kNoFlag
  uint32_t pad[2];
};
static_assert(sizeof(DevOp) == 64, "DevOp must stay 64 bytes");
constexpr uint32_t kDstF32 = 1u, kDstBcast = 2u, kFinal = 4u;  // kFinal: processing phase applies (hooked schedules)
constexpr uint32_t kStageAhead = 8u;  // stage op that waits for nothing: may run before the previous launch has completed

struct DevWait {
  uint32_t flag;
  uint32_t need;
};

struct ExecParams {
  void* base[kNumSlots];
  // Op i of queue q sits at index i * n_queues + q (queues padded to the longest one), so a
  // CTA finds its first op from its block index alone and learns the queue length from that
  // op: no dependent load in front of the first descriptor.
  const DevOp* ops;
  uint32_t n_queues;
  const uint64_t* srcs;         // src_stride packed addresses per op (same order as ops)
  const DevWait* waits;         // wait_stride entries per op
  uint32_t src_stride, wait_stride;
  unsigned long long* flags;    // one 64-bit counter per flag, monotone across executes; null if the schedule has none
  unsigned long long* epoch;    // [0] executes completed, [1] CTAs finished in this execute, [2] CTAs started (double-buffered staging)
  int* status;                  // pl_devstatus_t words + abort word (comm-owned)
  unsigned long long* trace;    // optional: per op (topological index) [start, end] %globaltimer stamps
  // SM-window launches of the bulk-copy executor: one CTA per SM is launched, the CTAs on SMs
  // whose bit is clear in sm_mask return, the others claim queues through sm_state (null: plain launch)
  unsigned long long* sm_state;
  uint32_t sm_mask[5];
  // Double-buffered staging (PL_OPT_STAGE_AHEAD): launch i uses flag set and scratch half i mod 2
  uint32_t stage_ahead;         // 0 / 1
  uint32_t n_flags;             // flags per set
  unsigned long long scratch_half;  // bytes from a rank's first staging buffer to its second
  unsigned long long timeout_ns;
  int n_ranks;
  int stages;            // shared-memory ring depth of the TMA executor
  uint32_t stage_bytes;  // bytes per ring slot
  float out_scale;       // multiplies every final (element-typed) sum; 1 = plain sum
  uint32_t hook;         // PL_HOOK_* bits (host side: selects the kernel variant; device: what final ops do)
  uint32_t hints;        // L2 policy bits for bulk copies: 1 loads of the caller's inputs evict-first, 2 stores evict-first, 4 copy loads evict-last
  uint32_t overlap_launch;  // host side only: launch with the programmatic stream serialization attribute
  uint32_t bcast_copies;      // host side only: the schedule holds broadcast copy ops (register executor variant)
  uint32_t pipelined_reduce;  // host side only: every reduce op is plain (element-typed operands), use the 12-warp variant
};

// Parameters of the packet executor (layered one-shot all-reduce, see pl_datapath_packet.cu).
struct PacketParams {
  const void* in[PL_MAX_RANKS];
  void* out[PL_MAX_RANKS];
  void* pkt[PL_MAX_RANKS];      // per rank: two packet buffers (even / odd global layer), 2 * message bytes each
  unsigned long long* epoch;    // [0] executes completed, [1] CTAs finished in this execute
  int* status;                  // pl_devstatus_t words + abort word (comm-owned)
  unsigned long long* trace;    // optional: per op [start, end] %globaltimer stamps
  unsigned long long timeout_ns;
  unsigned long long units_per_rank;  // 16-byte vectors of one layer's message
  long long break_op;                 // test hook: index of an op whose polls can never be satisfied, -1 = none
  int n_ranks, n_layers, ctas_per_rank;
  float out_scale;
};

struct Policy {
  int n_ctas, threads, datapath, stages;
  int idle_first, idle_count;  // SM-window launch: SMs that sit out (count 0: plain launch); idle_count < 0: asked for "none" 
  uint32_t stage_bytes, slice_bytes;
  // automatic slicing (slice_bytes == 0): bounds of a slice
  uint32_t min_slice, max_slice;
};

struct Lowered {
  std::vector<HostOp> ops;  // topological order
  int n_flags = 0;
  std::vector<uint32_t> flag_need;  // signals per execute, per flag
  uint64_t scratch_per_rank[PL_MAX_RANKS] = {0};
  uint64_t in_bytes[PL_MAX_RANKS] = {0};
  uint64_t out_bytes[PL_MAX_RANKS] = {0};
  uint64_t aux_bytes[PL_MAX_RANKS] = {0};
  uint64_t message_bytes = 0;
  int n_layers = 1;
  int role_queues[4] = {0, 0, 0, 0};  // queues per rank reserved for each role (0 = roles unused)
  bool queues_preassigned = false;    // the lowering fixed op.queue itself (packet schedules)
  bool double_buffered = false;       // two staging buffers and flag sets, alternated by launch parity
};

struct BuildRequest {
  int R, dtype, coll, algo;
  uint64_t count_per_rank;
  uint64_t chunk_bytes;
  const uint64_t* counts_v;  // R*R for all-to-all-v, else null
  int n_layers;              // 0: single collective
  int root;                  // rooted collectives
  bool staged;               // stage through schedule-owned memory (ordinary application buffers)
  uint64_t staging_bytes;    // staging capacity per rank (0 = default)
  int packet_ctas_per_rank;  // > 0: layered all-reduce on the packet datapath with this many CTAs per rank
  uint32_t hook;             // PL_HOOK_* bits
  bool stage_ahead;          // PL_OPT_STAGE_AHEAD
  int tuned_push_ctas;       // > 0: grid that pl_comm_tune measured for pushed copies on the bulk-copy datapath
  int tuned_idle_first, tuned_idle_count;  // and the window of idle SMs it measured with it (count 0: plain launch)
  int sm_count;              // SMs of the communicator's GPU
  Policy pol;
};

// orchestrator (host only, no CUDA)
pl_status_t lower(const BuildRequest& rq, Lowered* out, std::string* err);
void assign_queues(Lowered* L, int R, int n_queues, bool by_level = false);
// Largest number of ops one rank has at the same depth of the flag-dependency graph: the
// queues per rank a latency-bound schedule can keep busy at once.
int level_width(const Lowered& L, int R);
// bulk_datapath: the schedule runs on the bulk-copy executor, where program order on one queue
// orders less than on the register executor (see validate()).
pl_status_t validate(const Lowered& L, int R, std::string* err, bool bulk_datapath);
Policy default_policy(const BuildRequest& rq, int max_resident_ctas);

}  // namespace pl
