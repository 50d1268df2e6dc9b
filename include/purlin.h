/*
 * purlin.h -- C ABI of the B200 collectives executor.
 *
 * The library follows the paper's split into semantics, orchestration and datapath
 * (Sec. 1, "three-layer design"; Sec. 3.1-3.3):
 *
 *   semantics      a collective is named by (consume op, input layout, output layout)
 *                  (Listing 1) -> pl_collective_t;
 *   orchestration  where and when chunks move: the host lowers a collective into a flat
 *                  list of chunk-granular copy / reduce / copy-reduce ops with wait and
 *                  signal edges (Sec. 3.2, Listing 2, Algorithm 1) -> pl_schedule_build*;
 *   datapath       how bytes move: one persistent sm_100a kernel interprets the per-CTA op
 *                  queues (Sec. 3.3, Listing 3, Algorithm 2) -> pl_execute.
 *
 * R logical ranks are R sets of buffers in ONE GPU's memory; every rank's buffers are
 * visible to every other rank, i.e. the executor is the paper's variant that skips the
 * staging copy because application buffers are already peer accessible (Sec. 3.2,
 * "SNAC omits staging"; Sec. 5 "-ZS").
 *
 * Conventions
 *   - Plain C99 ABI, opaque handles, every call returns pl_status_t (PL_OK == 0).
 *   - All buffer pointers handed to pl_execute / pl_moe_* are DEVICE pointers unless a
 *     parameter is documented as host memory.  The library never owns, frees or writes
 *     input buffers; inputs are const, so repeating an execute repeats its result.
 *   - Errors are found on the host before any launch.  The device never traps: a wait
 *     that exceeds the schedule's time limit records a pl_devstatus_t and the kernel
 *     returns (see pl_comm_status).
 *   - pl_execute enqueues exactly one kernel on `stream`; it allocates nothing, copies
 *     nothing and never synchronises.  A schedule may be executed any number of times
 *     (flags carry a device-resident epoch; nothing is reset between executes).
 *   - One stream at a time per schedule: two executes of the same schedule must not
 *     overlap on the GPU.  Executes of DIFFERENT schedules may overlap only if their grids
 *     together are co-resident (pl_schedule_info reports each grid): the CTAs of a launch
 *     wait on one another, so two launches that each hold part of the SMs could starve each
 *     other until the wait limit reports PL_ERR_TIMEOUT.  Issuing all executes on one stream
 *     is always safe.
 *   - `stream` is a cudaStream_t passed as void* (NULL = the legacy default stream).
 *   - A communicator belongs to the CUDA device that was current when it was created; its
 *     schedules and plans live there.  Every later call on it must be made with that device
 *     current, otherwise the call returns PL_ERR_INVALID_ARG and launches nothing.
 */
#ifndef PURLIN_H_
#define PURLIN_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

#define PL_MAX_RANKS 16
#define PL_MAX_SRC 16   /* sources of one reduce op */
#define PL_MAX_WAITS 16 /* flags one op may wait on */

typedef enum {
  PL_OK = 0,
  PL_ERR_INVALID_ARG = 1,
  PL_ERR_UNSUPPORTED = 2,
  PL_ERR_ALIGNMENT = 3,
  PL_ERR_OOM = 4,
  PL_ERR_CUDA = 5,
  PL_ERR_TIMEOUT = 6,
  PL_ERR_OVERSUBSCRIBED = 7,
  PL_ERR_INVALID_SCHEDULE = 8,
  PL_ERR_OVERFLOW = 9
} pl_status_t;

/* Element types.  Reductions convert each element to fp32, accumulate in fp32 and
 * convert once at the end (Sec. 3.3, Eq. "rank-order"); int32 sums wrap.  PL_U8 is
 * valid for copy-only collectives. */
typedef enum {
  PL_BF16 = 0,
  PL_F32 = 1,
  PL_I32 = 2,
  PL_U8 = 3,
  /* Internal, appears only in op dumps: partial sums of an fp32 reduction that travel
   * between ops (ring hops, tree levels) as a (sum, correction) pair of fp32 per element,
   * 8 bytes, stored in blocks of 4 sums followed by their 4 corrections.  Not a valid
   * communicator dtype. */
  PL_F32X2 = 4
} pl_dtype_t;

/* Collectives (Listing 1): reduce-scatter = reduce, scattered->packed; all-gather = copy,
 * packed->scattered; all-to-all = copy, scattered->transposed; all-to-all-v its runtime-
 * sized twin; all-reduce = compose<reduce-scatter, all-gather>. */
typedef enum {
  PL_ALLREDUCE = 0,
  PL_REDUCE_SCATTER = 1,
  PL_ALLGATHER = 2,
  PL_ALLTOALL = 3,
  PL_ALLTOALLV = 4,
  PL_ALLGATHERV = 5,      /* copy, packedV -> scatteredV: rank p contributes n[p] elements */
  PL_REDUCE_SCATTERV = 6, /* reduce, scatteredV -> packedV: rank k receives partition k of n[k] elements */
  /* Rooted collectives (the paper's Appendix B proposes them as layouts plus a Root role):
   * only the root produces (scatter, broadcast) or only the root consumes (gather, reduce). */
  PL_BROADCAST = 7,       /* compose<scatter, all-gather>: the root's buffer reaches every rank   */
  PL_REDUCE = 8,          /* compose<reduce-scatter, gather>: the sum reaches the root only       */
  PL_SCATTER = 9,         /* rank r receives partition r of the root's buffer                     */
  PL_GATHER = 10          /* the root receives every rank's contribution in rank order            */
} pl_collective_t;

/* Algorithms.
 *   PL_ALGO_DIRECT        every consumer pulls straight from the producers' buffers (small
 *                         all-gathers, whose working set sits in L2, are pushed instead: the
 *                         producer writes its contribution into every output).  For
 *                         all-reduce this is Algorithm 1 without the staging role: rank k
 *                         reduces partition k from all inputs into its own output,
 *                         publishes reduced(k, c), and every other rank copies that chunk.
 *   PL_ALGO_ONESHOT       all-reduce only: every rank reduces the whole message itself.
 *   PL_ALGO_DIRECT_FUSED  all-reduce only: the reducer of partition k writes the result
 *                         into all R outputs (no gather step, fewest bytes).
 *   PL_ALGO_RING          textbook ring; partial sums of bf16 data travel in fp32, of fp32
 *                         data as compensated fp32 pairs (PL_F32X2), of int32 data in int32.
 *   PL_ALGO_TREE          all-reduce only: binomial reduce to a root, binomial broadcast from it;
 *                         the root of chunk c is rank c mod R (rank 0 for a one-chunk message).
 * Ring and tree are not in the paper (its only pattern is the direct pull); they are the
 * classical algorithms the benchmark configurations name. */
typedef enum {
  PL_ALGO_RING = 0,
  PL_ALGO_TREE = 1,
  PL_ALGO_DIRECT = 2,
  PL_ALGO_ONESHOT = 3,
  PL_ALGO_DIRECT_FUSED = 4,
  /* The library's pick for the collective and size, from the measurements on B200 (R = 8):
   * all-reduce: one-shot up to 32 KiB per rank, direct-fused above (the fastest of the five at
   * every size from 4 KiB to 256 MiB); everything else: direct.  pl_schedule_info does not
   * report the pick; pl_schedule_dump shows the ops. */
  PL_ALGO_AUTO = 5
} pl_algo_t;

typedef enum { PL_OP_COPY = 0, PL_OP_REDUCE = 1, PL_OP_COPY_REDUCE = 2 } pl_op_kind_t;
typedef enum { PL_BUF_IN = 0, PL_BUF_OUT = 1, PL_BUF_SCRATCH = 2 } pl_buf_kind_t;
/* How an op body moves bytes (Sec. 3.3).  TMA = cp.async.bulk staged through a
 * shared-memory ring of `stages` slots of `stage_bytes` (Algorithm 2: prime / steady /
 * drain).  LDST = 128-bit register loads/stores, unrolled (the paper's register path). */
typedef enum {
  PL_DP_AUTO = 0,
  PL_DP_LDST = 1,
  PL_DP_TMA = 2,
  /* Sec. 3.2, "Specializing for latency": data travels as 16-byte packets of 8 bytes of payload
   * and an 8-byte tag written with one store; the consumer polls the packet itself, so there is
   * no separate flag, fence or acquire on the path.  Only for pl_schedule_build_layers with
   * PL_ALGO_ONESHOT (or PL_ALGO_AUTO) and small messages (at most 128 KiB per rank; meant for
   * up to 64 KiB): rank r runs as a thread-block cluster of n_ctas / R CTAs (1, 2, 4 or 8; the
   * library picks 1 up to 4 KiB, else up to 8) that joins with a cluster barrier (a CTA barrier
   * for one CTA) when its layer's output is complete and then publishes its next contribution; the schedule owns two packet buffers per rank, alternated by layer
   * parity (Sec. 4.2, epoch-parity double buffering), tags are global layer numbers that only
   * grow, nothing is reset between executes.  pl_schedule_dump shows the same data movement
   * with the ordering rules as logical flags (no flag words exist on the device). */
  PL_DP_PACKET = 3
} pl_datapath_t;

typedef struct pl_comm_s* pl_comm_t;
typedef struct pl_schedule_s* pl_schedule_t;
typedef struct pl_moe_plan_s* pl_moe_plan_t;

/* Tuning knobs of one schedule ("codesign policy", Sec. 3.2/3.3).  Zero = take the
 * library's sm_100a default for the message size.  struct_size must be sizeof(). */
typedef struct {
  uint32_t struct_size;
  int32_t n_ctas;        /* persistent CTAs = op queues; rounded down to a multiple of R  */
  int32_t threads;       /* threads per CTA of the register datapath (multiple of 32, <=  */
                         /* 512); the bulk-copy datapath fixes its own (608, or 480 for   */
                         /* schedules of plain reduce ops: see pl_sched_info_t.threads)   */
  int32_t datapath;      /* pl_datapath_t                                                 */
  int32_t stages;        /* shared-memory ring depth S of the TMA pipeline                */
  uint32_t stage_bytes;  /* bytes per ring slot B_stage (multiple of 16)                  */
  uint32_t slice_bytes;  /* a chunk larger than this is split into slices run by several  */
                         /* CTAs; the chunk's flag then counts slices (Sec. 3.2, "last    */
                         /* staging CTA ... announces")                                   */
  uint64_t timeout_ns;   /* bound of every device-side wait; 0 = 2 s                      */
  uint32_t flags;        /* PL_OPT_*                                                      */
  uint64_t staging_bytes; /* PL_OPT_STAGED: staging capacity per rank; 0 = min(256 MiB, need) */
  float out_scale;       /* processing hook (Sec. 3.3, "processing phase ... while resident in   */
                         /* registers"): every final sum is multiplied by this in fp32 before   */
                         /* the one conversion to the element type, e.g. 1/R for an average.    */
                         /* 0 = no scaling.  Float element types only (PL_ERR_UNSUPPORTED).     */
  uint32_t hook;         /* PL_HOOK_* bits: further steps of the processing phase (below)        */
  int32_t idle_sm_first; /* SM-window launch (bulk-copy datapath, schedules without flags): one  */
  int32_t idle_sm_count; /* CTA per SM is launched and the CTAs on SMs idle_sm_first ..          */
                         /* idle_sm_first + idle_sm_count - 1 return at once; the others claim   */
                         /* the queues.  n_ctas must be 0 or the SM count minus idle_sm_count,   */
                         /* which must be a multiple of R.  0 = the library decides (a plain     */
                         /* launch, or the window pl_comm_tune measured / the default one for    */
                         /* pushed all-gathers).  Which SMs take part decides how fast a write-  */
                         /* dominated stream runs (pl_comm_tune).  PL_ERR_UNSUPPORTED where it   */
                         /* does not apply (flags, register or packet datapath, more than one    */
                         /* CTA per SM, PL_OPT_OVERLAP_LAUNCH: the claim words serve one launch  */
                         /* at a time).  No counterpart in the paper.                            */
} pl_sched_opts_t;
/* The processing phase as a small family (Sec. 3.3: the phase between the last addition and the
 * store is configurable while the sum sits in registers).  With s = out_scale (1 if unset):
 *   out_r[i] = cvt( s * sum_p x_p[i]  [+ aux_r[i]] )
 * PL_HOOK_RESIDUAL  adds a second operand per rank, aux[r] (pl_bufs_t), laid out like out[r] and
 *                   of the element type, in fp32 before the one conversion (the residual
 *                   connection that follows a tensor-parallel all-reduce).
 * PL_HOOK_F32_OUT   bf16 schedules only: no conversion, out[r] holds fp32 (twice the bytes;
 *                   pl_schedule_info reports them).
 * Both need a collective whose outputs are written by its reduce ops and by nothing else:
 * reduce-scatter (direct, ring, staged), one-shot and direct-fused all-reduce (also layered),
 * reduce-scatter-v, rooted reduce.  Collectives that finish with a copy phase (ring / tree /
 * two-shot all-reduce) return PL_ERR_UNSUPPORTED: a copied result cannot differ per rank.
 * Float element types only; not on the packet datapath. */
#define PL_HOOK_RESIDUAL 1u
#define PL_HOOK_F32_OUT 2u
#define PL_OPT_SKIP_VALIDATE 1u /* do not run the static validator inside build */
/* Treat in/out as ORDINARY application buffers that peers must not touch (Sec. 3.2, "Protocol
 * operations": stage -> notify -> consume; Algorithm 1 with its staging role).  Every rank
 * first copies its contribution chunk by chunk into schedule-owned staging memory and
 * publishes staged(r,k,c); consumers pull only from staging; a composed all-reduce also keeps
 * its reduced chunks Y_k[c] in staging and the gather role publishes consumed(r,k,c).  Staging
 * holds staging_bytes per rank: when the message needs more, chunk slots are reused cyclically
 * (Sec. 4.1) and a stage op waits until the slot's previous chunk has been consumed.  Only
 * PL_ALGO_DIRECT.  One staging buffer per rank, unless PL_OPT_STAGE_AHEAD asks for the paper's
 * two buffers alternated by epoch parity. */
#define PL_OPT_STAGED 4u
/* Record, for every op, when its waits were satisfied and when its signal was about to be
 * released (%globaltimer, ns) into a schedule-owned buffer: see pl_schedule_trace_read. */
#define PL_OPT_TRACE 8u
/* Launch pl_execute's kernel with CUDA's programmatic stream serialization attribute, so that
 * when the kernel in front of it on the stream is another execute, its CTAs may be set up
 * while that one drains (the kernel waits for the completion of everything in front of it
 * before it reads anything an earlier launch wrote, so stream order is kept as seen by the
 * data).  Shortens back-to-back executes; no effect after any other kind of work.  The paper
 * has no counterpart (it measures calls inside a CUDA graph, Sec. 5). */
#define PL_OPT_OVERLAP_LAUNCH 16u
/* Epoch-parity double buffering of the staging memory (Sec. 4.1-4.2: two staging buffers
 * alternated by the parity of a persistent epoch, so that a rank can enter call n+1 while peers
 * still consume call n).  Needs PL_OPT_STAGED and PL_OPT_OVERLAP_LAUNCH.  The schedule owns two
 * staging buffers and two flag sets per rank; launch i uses set i mod 2 (the launch number is a
 * device-resident counter taken at kernel entry, so CUDA-graph replays stay consistent).  The
 * stage role of execute n+1 -- the leading stage ops of a queue that wait for nothing: they only
 * read the caller's inputs and write the other staging buffer -- runs BEFORE the kernel waits for
 * execute n to complete; everything else runs after it.  The caller promises that the inputs of
 * an execute are not written by the launch directly in front of it on the stream (an execute
 * that consumes the previous execute's outputs must not use this option).  The paper advances
 * its epoch by the chunk count rounded to an odd number so that the parity flips on every call;
 * here the launch counter itself is the epoch and its lowest bit the parity. */
#define PL_OPT_STAGE_AHEAD 32u
#define PL_OPT_NO_L2_HINTS 2u  /* bulk copies without L2 eviction hints (default: stores evict-first,
                                  sources of copy ops evict-last) */
/* The caller's input buffers are read here for the last time (gradients that the reduce-scatter
 * consumes, the partition an all-gather spreads): the bulk-copy datapath then loads them with an
 * L2 evict-first hint, so that the stream of inputs displaces itself from L2 and not what this
 * launch writes or what the launch behind it is about to read.  Measured on the reduce-scatter ->
 * all-gather step (8 x 64 MiB): the all-gather finds the reduce-scatter's 64 MiB of results in L2
 * (6 MB of DRAM reads instead of 67 MB) and the step takes 5 % less; a launch repeated on its own
 * is 1-2 % slower with the hint, which is why it is not the default.  Ignored by schedules that
 * read an input byte more than once (one-shot all-reduce), by the register and packet datapaths
 * and together with PL_OPT_NO_L2_HINTS.  Nothing in the paper corresponds to this option (its
 * inputs live in other GPUs' memories). */
#define PL_OPT_INPUTS_LAST_USE 64u

/* A buffer reference inside an op: rank's in/out/scratch buffer, byte offset, and the
 * element type stored there (partials of a bf16 reduction are PL_F32). */
typedef struct {
  int32_t rank;
  int32_t buf;   /* pl_buf_kind_t */
  int32_t dtype; /* pl_dtype_t */
  int32_t pad_;
  uint64_t offset; /* bytes */
} pl_ref_t;

/* One op of a schedule as reported by pl_schedule_dump (host copy, for inspection and
 * for replaying a schedule on the CPU in tests). */
typedef struct {
  int32_t kind;      /* pl_op_kind_t */
  int32_t exec_rank; /* rank whose CTAs run the op (the consumer that pulls) */
  int32_t queue;     /* CTA / op queue the op is placed on */
  int32_t topo;      /* position in the global topological order */
  int32_t layer;     /* layer of a multi-layer schedule, else 0 */
  int32_t n_src;
  int32_t n_wait;
  int32_t signal_flag; /* flag incremented (release) when the op's writes are done, -1 none */
  int32_t signal_flag2;/* optional second flag incremented the same way, -1 none */
  int32_t dst_bcast;   /* 1: dst is replicated at the same offset into out[0..R); 3: and the op is final */
                       /* bit 1 (value 2): the op writes final output and runs the processing phase    */
                       /* bit 2 (value 4): stage op that PL_OPT_STAGE_AHEAD may run before the launch  */
                       /* in front has completed                                                       */
  uint64_t count;      /* elements; COPY ops count bytes (dtype PL_U8) */
  pl_ref_t dst;
  pl_ref_t src[PL_MAX_SRC];
  int32_t wait_flag[PL_MAX_WAITS];
  uint32_t wait_need[PL_MAX_WAITS]; /* signals per execute the flag must have received */
} pl_op_t;

typedef struct {
  uint64_t n_ops, n_queues, n_flags, n_waits, n_layers;
  uint64_t bytes_read, bytes_written;  /* summed over ops: the schedule's algorithmic bytes */
  uint64_t message_bytes;              /* per-rank message size in the paper's convention  */
                                       /* (Sec. 5: gathered output for all-gather, per-rank */
                                       /* input otherwise)                                  */
  uint64_t scratch_bytes;              /* device scratch the schedule owns (all ranks)      */
  uint64_t in_bytes[PL_MAX_RANKS];     /* bytes pl_execute requires in bufs->in[r]          */
  uint64_t out_bytes[PL_MAX_RANKS];    /* bytes pl_execute requires in bufs->out[r]         */
  int32_t grid, threads, smem_bytes, datapath, stages;
  uint32_t stage_bytes, slice_bytes;
  uint64_t aux_bytes[PL_MAX_RANKS];    /* bytes pl_execute requires in bufs->aux[r] (PL_HOOK_RESIDUAL) */
  int32_t out_dtype;                   /* element type stored in out[r]: PL_F32 under PL_HOOK_F32_OUT  */
  uint32_t hook;                       /* PL_HOOK_* bits of the schedule                               */
  uint64_t hbm_bytes;                  /* bytes that must cross the memory interface when nothing is   */
                                       /* cached between launches: bytes_read with every byte of the   */
                                       /* caller's inputs (and second operands) counted once, however  */
                                       /* many ops read it, plus bytes_written                         */
  int32_t idle_sm_first, idle_sm_count; /* SM-window launch: the SMs that sit out (count 0: plain launch of `grid` CTAs) */
} pl_sched_info_t;

/* Device buffers of one execute: in[r] / out[r] for r < R, 16-byte aligned, non-overlapping.
 * aux[r] is only read by schedules built with PL_HOOK_RESIDUAL (second operand of the
 * processing phase, laid out like out[r]); it may overlap nothing that is written. */
typedef struct {
  const void* in[PL_MAX_RANKS];
  void* out[PL_MAX_RANKS];
  size_t in_bytes[PL_MAX_RANKS];
  size_t out_bytes[PL_MAX_RANKS];
  const void* aux[PL_MAX_RANKS];
  size_t aux_bytes[PL_MAX_RANKS];
} pl_bufs_t;

/* Device-side status record (first writer wins).  code == PL_OK when nothing happened. */
typedef struct {
  int32_t code;   /* PL_OK or PL_ERR_TIMEOUT */
  int32_t queue;  /* CTA that gave up */
  int32_t op;     /* index of the op inside the schedule (topological index) */
  int32_t flag;   /* flag it was waiting on */
  uint64_t expected, observed;
} pl_devstatus_t;

/* ---- communicator ------------------------------------------------------------------ */

/* The communicator holds the state that outlives one call (Sec. 4.2: the paper's executor keeps
 * persistent per-communicator state -- epoch, flags, staging -- between calls so that nothing is
 * set up or cleared per collective): here the device status record and the list of schedules,
 * each of which owns its epoch and flag words.
 *
 * Create a communicator of R emulated ranks (2 <= R <= PL_MAX_RANKS) with element type
 * `dtype` on the CURRENT CUDA device.  Allocates a few device words (status, abort).
 * Errors: PL_ERR_INVALID_ARG (R, dtype, out), PL_ERR_CUDA (no usable device). */
pl_status_t pl_comm_create(int R, pl_dtype_t dtype, pl_comm_t* out);

/* Same, but host-only: schedules can be built, validated, inspected and dumped; nothing is
 * placed on a device and pl_execute returns PL_ERR_UNSUPPORTED.  Needs no GPU. */
pl_status_t pl_comm_create_planner(int R, pl_dtype_t dtype, pl_comm_t* out);

/* Destroy a communicator.  Its schedules and plans must be destroyed first
 * (PL_ERR_INVALID_ARG otherwise). */
pl_status_t pl_comm_destroy(pl_comm_t comm);

/* Measure, on this communicator's GPU, with how many CTAs and on WHICH SMs the write-dominated
 * direct schedules of the bulk-copy datapath (all-gather, all-gather-v, broadcast: 1 read : R
 * writes) run fastest, and make the result the default of later builds on this communicator
 * (opts.n_ctas / opts.idle_sm_count still override; schedules already built keep theirs).  Such
 * a stream is served best with fewer than all SMs writing, and with the right ones sitting out:
 * 16-20 idle SMs taken from SM ids 0-31 or 64-79 gave 97-103 us for the 8 x 64 MiB all-gather on
 * every B200 tried, the same number anywhere else 108-116 us; which SMs a plain launch of fewer
 * CTAs leaves idle is up to the hardware and differs from one GPU to the next of the same model
 * (plain launches: 101 us at best on some, 107 us on others).  Candidates: plain launches of
 * every multiple of R between 3/4 of the resident CTAs and all of them, and the same grids
 * launched as one CTA per SM with the idle SMs as a window starting at SM 0, 8, 16 or 64; each
 * runs an all-gather of 64 MiB behind the reduce-scatter that produces its input, both with
 * PL_OPT_INPUTS_LAST_USE (2 + 10 pairs of launches; a candidate replaces the pick only if it is
 * 0.5 % faster, so equal ones resolve to the larger grid and the plain launch): where an all-gather usually runs, its input
 * is in L2 and its DRAM traffic almost purely writes, and the fastest candidate is not always the
 * one that is fastest alone.  Runs on `stream`, on buffers this call allocates and frees
 * ((2 R + 1) x 64 MiB).  Synchronises: a call for set-up time, not for the hot path.  Nothing
 * in the paper corresponds to it.  The outputs (each may be NULL) receive the chosen grid and
 * window (count 0: a plain launch).
 * Errors: PL_ERR_UNSUPPORTED (planner communicator), PL_ERR_OOM, PL_ERR_CUDA, PL_ERR_INVALID_ARG
 * (the current device is not the communicator's). */
pl_status_t pl_comm_tune(pl_comm_t comm, void* stream, int32_t* push_ctas_out, int32_t* idle_sm_first_out,
                         int32_t* idle_sm_count_out);

/* Read the device status record as it stands at the time of the call (on an internal stream: the
 * call waits for no other work, so synchronise the stream of the executes you ask about first).
 * Returns PL_OK and fills *out; out->code tells whether a wait timed out since the last reset. */
pl_status_t pl_comm_status(pl_comm_t comm, pl_devstatus_t* out);

/* Clear the status record and re-zero the flags and epochs of every schedule of `comm`
 * (asynchronously on `stream`).  Required after a timeout before executing again. */
pl_status_t pl_comm_reset(pl_comm_t comm, void* stream);

/* Text of the last build or validation failure on this communicator ("" if none): which
 * rule of the size / algorithm / schedule checks was violated.  The pointer stays valid until
 * the next failing call on the same communicator. */
const char* pl_comm_last_error(pl_comm_t comm);

/* ---- orchestration ----------------------------------------------------------------- */

/* Lower a fixed-size collective into a schedule.
 *   count_per_rank  elements of the per-rank message: the INPUT element count for
 *                   all-reduce, reduce-scatter and all-to-all; the per-rank CONTRIBUTION
 *                   for all-gather (output = R * count_per_rank).
 *   chunk_bytes     chunk size in bytes of the element type (multiple of 16); clipped to
 *                   the partition size; the last chunk of a partition may be short.  It is
 *                   the granularity of the flags; a schedule whose ops neither wait nor
 *                   signal (direct all-gather) may be cut into smaller chunks.
 * Partitioned collectives need count_per_rank * elem_size divisible by R*16
 * (PL_ERR_INVALID_ARG).  PL_ERR_UNSUPPORTED for algorithm/collective pairs that do not
 * exist (tree, one-shot and fused are all-reduce only; PL_U8 cannot be reduced).
 * PL_ERR_OVERSUBSCRIBED when the requested CTAs cannot all be co-resident (the executor
 * spins on flags, so every queue must be running).  PL_ERR_OOM / PL_ERR_CUDA on device
 * allocation failure.  The schedule owns its device op list, flags and scratch. */
pl_status_t pl_schedule_build(pl_comm_t comm, pl_collective_t coll, pl_algo_t algo,
                              size_t count_per_rank, size_t chunk_bytes,
                              const pl_sched_opts_t* opts, pl_schedule_t* out);

/* Variable-size collectives (Listing 1's V namings; partition sizes given at run time).
 * counts is a HOST array in elements:
 *   PL_ALLTOALLV        R*R entries, row-major [src][dst];
 *   PL_ALLGATHERV       R entries: n[p] = contribution of rank p (output = their concatenation);
 *   PL_REDUCE_SCATTERV  R entries: n[k] = partition k of every rank's input, reduced to rank k.
 * Every size times elem_size must be a multiple of 16 (PL_ERR_ALIGNMENT); zero is allowed.
 * PL_ALGO_DIRECT only.  The reported message size is the total T (as the paper plots it). */
pl_status_t pl_schedule_build_v(pl_comm_t comm, pl_collective_t coll, pl_algo_t algo,
                                const size_t* counts, size_t chunk_bytes,
                                const pl_sched_opts_t* opts, pl_schedule_t* out);

/* Rooted collectives, root given at run time (0 <= root < R).  count_per_rank: the root's
 * message for PL_BROADCAST (every output has that size) and the per-rank message for PL_REDUCE
 * (the root's output has that size); the per-rank partition for PL_SCATTER (root input =
 * R * count) and PL_GATHER (root output = R * count).  Ranks that contribute nothing need no
 * input buffer and ranks that receive nothing no output buffer (pl_schedule_info reports 0
 * bytes for them).  Broadcast and reduce are the two-step compositions the paper names, in one
 * launch: for broadcast rank k pulls partition k from the root and publishes it, every rank
 * then pulls partition k from rank k; for reduce rank k reduces partition k into schedule-owned
 * memory (the root straight into its output) and the root gathers.  Message bytes divisible by
 * 16*R for broadcast and reduce, by 16 for scatter and gather.  PL_ALGO_DIRECT only. */
pl_status_t pl_schedule_build_rooted(pl_comm_t comm, pl_collective_t coll, int root, size_t count_per_rank,
                                     size_t chunk_bytes, const pl_sched_opts_t* opts, pl_schedule_t* out);

/* n_layers back-to-back all-reduces in ONE launch (the latency path: no kernel launch,
 * memset or host round trip per layer).  The shape is tensor-parallel decoding (Sec. 2.1:
 * decode exchanges messages of tens of KB per layer, where set-up and synchronisation cost
 * dominate; Sec. 3.2 "Specializing for latency").  Layer l reads in[r] + l*M and writes out[r] + l*M
 * (M = count_per_rank * elem_size).  Rank r's layer-(l+1) contribution counts as published
 * only when r's layer-l output is complete, and no consumer reads it earlier.  Algorithms:
 * PL_ALGO_ONESHOT, PL_ALGO_DIRECT, PL_ALGO_DIRECT_FUSED; PL_ALGO_AUTO picks direct-fused on the
 * register executor, and for messages of at most 4 KiB (with grid, datapath and hooks left to the
 * library) one-shot on the packet datapath with one CTA per rank, the fastest form there. */
pl_status_t pl_schedule_build_layers(pl_comm_t comm, pl_algo_t algo, size_t count_per_rank,
                                     int n_layers, const pl_sched_opts_t* opts,
                                     pl_schedule_t* out);

pl_status_t pl_schedule_info(pl_schedule_t s, pl_sched_info_t* out);

/* Copy up to `cap` ops (topological order) into `ops`; *n receives the total op count.
 * ops may be NULL to query the count. */
pl_status_t pl_schedule_dump(pl_schedule_t s, pl_op_t* ops, size_t cap, size_t* n);

/* Static check of a schedule (also run by build unless PL_OPT_SKIP_VALIDATE): every output
 * byte written exactly once, every read of a byte the schedule writes is ordered after that
 * write by a wait edge (or by queue order), every flag's signals precede its waiters in
 * the topological order, queue order embeds in that order.  On failure returns
 * PL_ERR_INVALID_SCHEDULE and writes a message into msg (may be NULL). */
pl_status_t pl_schedule_validate(pl_schedule_t s, char* msg, size_t msg_cap);

/* Copy the trace of the LAST execute to a HOST array of 2 * n_ops entries (index 2*i = start of
 * op i in topological order: the moment its waits were satisfied; 2*i+1 = end: the moment just
 * before its signal was released; the bulk-copy executor stamps the end only for ops that
 * signal, others read 0).  Needs PL_OPT_TRACE at build (PL_ERR_INVALID_ARG otherwise).
 * Synchronises `stream`.  Useful to see where a schedule's time goes and to check on the real
 * device that every waiter started after all of its signallers ended. */
pl_status_t pl_schedule_trace_read(pl_schedule_t s, uint64_t* out, size_t cap_entries, void* stream);

/* TEST HOOK: remove the first wait edge of op `op_index` from the host copy of the schedule,
 * so that pl_schedule_validate can be shown to notice the missing ordering.  The device copy
 * is left alone; do not execute the schedule afterwards. */
pl_status_t pl_schedule_debug_drop_wait(pl_schedule_t s, size_t op_index);

/* TEST HOOK: corrupt one wait edge of a built schedule so that it can never be satisfied
 * (raises the needed count of op `op_index`'s first wait).  Used with a short timeout_ns to
 * exercise the bounded-wait path without hanging a GPU. */
pl_status_t pl_schedule_debug_break_wait(pl_schedule_t s, size_t op_index);

pl_status_t pl_schedule_destroy(pl_schedule_t s);

/* ---- datapath ---------------------------------------------------------------------- */

/* Run the schedule once over `bufs` on `stream` (asynchronous, one kernel launch): the datapath
 * tier (Sec. 3.3, Listing 3 and Algorithm 2): every CTA walks its op queue, and per op waits,
 * moves the chunk through the pipeline with the op's consume step (copy or rank-ordered
 * reduce, Eq. "rank-order") and signals.
 * Errors (all before launch): PL_ERR_INVALID_ARG (NULL pointer, buffer smaller than
 * pl_schedule_info reports, in/out ranges that overlap), PL_ERR_ALIGNMENT (a pointer not
 * 16-byte aligned), PL_ERR_UNSUPPORTED (planner communicator), PL_ERR_CUDA (launch). */
pl_status_t pl_execute(pl_schedule_t s, const pl_bufs_t* bufs, void* stream);

/* End-to-end form for callers whose data lives in HOST memory: copies host->in[r] into
 * dev->in[r] (cudaMemcpyAsync on `stream`; pinned memory makes it truly asynchronous), runs
 * the schedule, and copies dev->out[r] back into host->out[r].  `dev` supplies the device
 * staging buffers (caller-owned).  Sizes come from pl_schedule_info. */
pl_status_t pl_execute_host(pl_schedule_t s, const pl_bufs_t* host, const pl_bufs_t* dev,
                            void* stream);

/* Pipelined form of pl_execute_host for a sequence of host executes on one communicator (no
 * counterpart in the paper, whose data never leaves the GPUs): the uploads run on an upload
 * stream of the communicator, the schedule on `stream`, the downloads on a download stream, tied
 * together by events, so that the download of one call overlaps the upload of the next (the host
 * link carries both directions at once).  What is ordered: an upload waits for the schedule of
 * the previous async host execute (which read the device inputs it overwrites) and for every
 * download still in flight that writes a host range it reads or reads a device range it
 * overwrites; the schedule waits for its uploads and for every download that still reads device
 * outputs it overwrites; downloads run in call order.  What is NOT ordered: other work the caller
 * puts on `stream` between two async host executes is waited for only by the first call and
 * after a change of stream, so the device staging buffers in `dev` must not be touched by such
 * work; and `stream` does not wait for the downloads: the host outputs are complete after
 * pl_comm_host_sync (host blocks) or behind pl_comm_host_fence (the given stream waits).
 * Allocates nothing after the first call (two streams and a fixed set of events).  Arguments and
 * errors as pl_execute_host. */
pl_status_t pl_execute_host_async(pl_schedule_t s, const pl_bufs_t* host, const pl_bufs_t* dev,
                                  void* stream);
/* Bytes the host entry points of this communicator have copied so far, host to device and
 * device to host (either pointer may be NULL).  pl_execute_host_async does not upload an input
 * that is already on the device: when a call's host input buffer is exactly the host output
 * buffer of the immediately preceding call, that call's download is still in flight, and the
 * device input buffer is the device buffer that download reads (a reduce-scatter's result handed
 * to an all-gather through a host buffer), the bytes are the ones the previous schedule left
 * there, and neither copy nor wait is needed. */
pl_status_t pl_comm_host_stats(pl_comm_t comm, uint64_t* h2d_bytes, uint64_t* d2h_bytes);
/* Make `stream` wait (asynchronously) for all downloads of earlier pl_execute_host_async calls. */
pl_status_t pl_comm_host_fence(pl_comm_t comm, void* stream);
/* Block the calling thread until all downloads of earlier pl_execute_host_async calls are done. */
pl_status_t pl_comm_host_sync(pl_comm_t comm);

/* ---- MoE expert-parallel dispatch / combine (all-to-all-v of token rows) ------------ */

/* Plan for R ranks x tokens_per_rank tokens of `hidden` elements (comm dtype, row bytes a
 * multiple of 16), n_experts experts (n_experts % R == 0, expert e lives on rank
 * e / (n_experts/R)), topk distinct experts per token (topk <= 32).  recv_capacity_rows =
 * rows each rank's receive buffer can hold.  The plan owns device scratch for counts,
 * offsets and the row positions that combine reuses. */
pl_status_t pl_moe_plan_create(pl_comm_t comm, int tokens_per_rank, int hidden, int n_experts,
                               int topk, size_t recv_capacity_rows, pl_moe_plan_t* out);
pl_status_t pl_moe_plan_destroy(pl_moe_plan_t plan);

/* Dispatch (Table 2, expert parallelism: scatteredV -> transposedV).  Host arrays of R
 * DEVICE pointers: x[p] rows [T][hidden]; topk_idx[p] int32 [T][topk]; recv[r] rows
 * [recv_capacity_rows][hidden]; recv_meta[r] int32 [recv_capacity_rows][4] =
 * (source rank, token, slot, expert) per received row (may be NULL to skip).
 * One row is sent per (token, slot); rank r receives rows ordered by (source rank,
 * expert, token).  Counts and offsets are computed on the device (histogram + exclusive
 * scans).  Rows beyond recv_capacity_rows are dropped and flagged (pl_moe_plan_read
 * returns PL_ERR_OVERFLOW). */
pl_status_t pl_moe_dispatch(pl_moe_plan_t plan, const void* const* x,
                            const int32_t* const* topk_idx, void* const* recv,
                            int32_t* const* recv_meta, void* stream);

/* Combine: out[p][t][:] = sum_{j<topk} gates[p][t][j] * y[rank(e_j)][pos(p,t,j)][:] in fp32,
 * ascending j, one final conversion; y has the layout dispatch produced, pos is the row
 * dispatch wrote for (p,t,j).  Must follow a dispatch on the same plan (it reuses pos). */
pl_status_t pl_moe_combine(pl_moe_plan_t plan, const void* const* y, const float* const* gates,
                           void* const* out, void* stream);

/* Combine with the gates computed on the GPU: logits[p] holds, per token, the K logits of
 * the selected experts (fp32 [T][topk], slot order); the kernel takes their softmax in fp32
 * (maximum subtracted) and uses the result as gates.  Otherwise as pl_moe_combine. */
pl_status_t pl_moe_combine_logits(pl_moe_plan_t plan, const void* const* y, const float* const* logits,
                                  void* const* out, void* stream);

/* Synchronise `stream` and copy the plan's bookkeeping to HOST arrays (any may be NULL):
 * pos int32 [R][T][topk]; counts int64 [R][R] rows src->dst; expert_counts int64
 * [R][n_experts].  Returns PL_ERR_OVERFLOW if the last dispatch dropped rows. */
pl_status_t pl_moe_plan_read(pl_moe_plan_t plan, int32_t* pos, int64_t* counts,
                             int64_t* expert_counts, void* stream);

/* ---- for callers that cannot allocate ------------------------------------------------ */

/* Ring reduce-scatter with no allocation of any kind (the paper has no counterpart; this
 * entry point exists for deployments, not for the method).
 *
 * Who needs it: code that must not call cudaMalloc where the collective happens -- a
 * serving loop that cannot afford cudaMalloc's device-wide synchronisation, a component
 * living under a pre-planned memory arena, a plugin that only ever receives buffers.  The
 * schedule-based path (pl_schedule_build + pl_execute) allocates its op list, flags and the
 * scratch for travelling partial sums at build time; this call instead keeps the partial
 * sums in a fixed 32 MiB array that is part of the library image on every GPU that loads
 * the library (it stays resident until the process exits), and launches exactly one kernel.
 *
 *   in[r]   DEVICE pointer, count_per_rank elements (R partitions), 16-byte aligned
 *   out[r]  DEVICE pointer, count_per_rank / R elements: sum over ranks of partition r
 *   status  optional DEVICE word owned by the caller: cleared on `stream` before the launch,
 *           set to PL_ERR_TIMEOUT if a wait inside the kernel gave up (2 s); may be NULL
 * in / out are HOST arrays of R pointers.  dtype: PL_BF16, PL_F32 or PL_I32; results are the
 * same as the ring reduce-scatter schedule's (fp32 partial sums for bf16, compensated pairs
 * for fp32, ascending ring order).
 *
 * Limits and rules
 *   - R * (R-2) * (count_per_rank / R) * partial_size must fit the 32 MiB array (partial_size
 *     4 bytes for bf16 and int32, 8 for fp32); larger messages return PL_ERR_OVERFLOW before
 *     anything is launched.  Other errors as pl_schedule_build / pl_execute
 *     (PL_ERR_INVALID_ARG, PL_ERR_ALIGNMENT, PL_ERR_UNSUPPORTED, PL_ERR_CUDA).
 *   - The first call on a device looks up the device address of the built-in array (a one-
 *     time set-up with that device current); make that first call outside any stream capture.
 *   - All calls on a GPU share the array, and it keeps whatever the last call left there.
 *     Nothing in it needs clearing between calls (the kernel numbers its calls with a counter
 *     that lives on the device and ignores readiness marks of earlier calls, also after a
 *     time-out), but two calls that overlap in time on the same GPU (e.g. on two streams) race
 *     on it: issue them on one stream or order them.
 *   - Calls no cudaMalloc, cudaFree or other allocating routine. */
pl_status_t pl_reduce_scatter_ring_static(int R, pl_dtype_t dtype, size_t count_per_rank,
                                          const void* const* in, void* const* out,
                                          int32_t* status, void* stream);

/* TEST HOOK for the call above (the paper has no counterpart): same arguments, but every wait
 * inside the kernel expects a mark that is never published and gives up after timeout_ns
 * (1 ns .. 1 s), so that *status becomes PL_ERR_TIMEOUT and the outputs are incomplete.  Shows
 * that a time-out leaves the GPU and the built-in array usable for the next call. */
pl_status_t pl_reduce_scatter_ring_static_debug_timeout(int R, pl_dtype_t dtype, size_t count_per_rank,
                                                        const void* const* in, void* const* out,
                                                        int32_t* status, void* stream, uint64_t timeout_ns);

/* Deduplicated variant (one row per token and DESTINATION RANK instead of per expert: when
 * several of a token's experts live on one rank the row crosses once; 32 % fewer rows on the
 * Zipf(1.2) top-8 workload).  Same plan, same argument conventions as pl_moe_dispatch.
 * Rank r receives rows in (source rank, token) order; recv_meta row = (source rank, token,
 * slot mask, r) where bit j of the mask says that slot j's expert lives on r.
 * recv_capacity_rows bounds these rows as well. */
pl_status_t pl_moe_dispatch_dedup(pl_moe_plan_t plan, const void* const* x, const int32_t* const* topk_idx,
                                  void* const* recv, int32_t* const* recv_meta, void* stream);

/* Reverse of the deduplicated dispatch: every rank returns ONE row per received row (its
 * expert layer has applied the gates and summed its local experts);
 * out[p][t][:] = sum over destination ranks r, ascending, of z[r][pos(p,t,r)][:] in fp32 with
 * one final conversion (bf16 only). */
pl_status_t pl_moe_combine_dedup(pl_moe_plan_t plan, const void* const* z, void* const* out, void* stream);

/* Bookkeeping of the last deduplicated dispatch, to HOST arrays (may be NULL): pos int32
 * [R][T][R] = row of (p, t) at rank r or -1; counts int64 [R][R].  Synchronises `stream`. */
pl_status_t pl_moe_plan_read_dedup(pl_moe_plan_t plan, int32_t* pos, int64_t* counts, void* stream);

/* ---- diagnostic: stream ceilings of the bulk-copy machinery ------------------------ */

/* NOT PART OF THE PAPER'S METHOD.  Enqueues one kernel on `stream` that streams `bytes` with
 * the instructions the executors use (bulk asynchronous copies through a shared-memory ring,
 * one CTA per SM): kind 0 reads src and drops the data, kind 1 fills dst with a fixed pattern
 * (32-bit word j of every 32 KiB tile = j * 2654435761 mod 2^32), kind 2 copies src to dst,
 * kind 3 writes every tile of src to the same offset of 8 consecutive regions of dst (one read
 * to eight writes; on a 148-SM part 132 CTAs work and SMs 8-23 sit out, the kind of SM window the
 * write-dominated schedules use: kind-3 probes must not run concurrently with one another, they
 * share the window's claim words).  Timed with CUDA events by the caller it gives the pure-read, pure-write,
 * copy and 1:8 bandwidth that bound the read-dominated (reduce-scatter, MoE combine), balanced
 * (all-to-all) and write-dominated (all-gather, MoE dispatch) collectives on this GPU.
 *   src, dst  DEVICE pointers, 16-byte aligned, `bytes` long (src unused for kind 1, dst for
 *             kind 0; dst 8 * bytes long for kind 3); bytes a positive multiple of 32768
 *   status    optional DEVICE word of the caller: cleared on `stream`, set to PL_ERR_TIMEOUT if
 *             a wait inside the kernel gave up (2 s); may be NULL
 * Errors (before any launch): PL_ERR_INVALID_ARG, PL_ERR_ALIGNMENT, PL_ERR_CUDA. */
pl_status_t pl_probe_hbm(int kind, const void* src, void* dst, size_t bytes, int32_t* status, void* stream);

const char* pl_status_string(pl_status_t st);

/* Number of kernels this library has launched in the calling process (all entry points). */
uint64_t pl_launch_count(void);

#ifdef __cplusplus
}
#endif
#endif /* PURLIN_H_ */
