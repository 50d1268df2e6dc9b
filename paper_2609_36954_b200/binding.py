"""ctypes binding of libpurlin.so: argument marshalling only.

Every function below maps 1:1 onto the C entry point of the same name declared in
``include/purlin.h``; all work (orchestration in host C++, datapath in CUDA) happens
inside the library.  Device buffers are passed as integer addresses (e.g.
``tensor.data_ptr()``); ``stream`` is a ``cudaStream_t`` handle as int (e.g.
``torch.cuda.current_stream().cuda_stream``).  There is no CPU fallback: if the
library is missing or a call fails, a ``PurlinError`` is raised.
"""
from __future__ import annotations

import ctypes as C
import os

from . import build as _build

PL_MAX_RANKS = 16
PL_MAX_SRC = 16
PL_MAX_WAITS = 16

# status
PL_OK, PL_ERR_INVALID_ARG, PL_ERR_UNSUPPORTED, PL_ERR_ALIGNMENT, PL_ERR_OOM, PL_ERR_CUDA, \
    PL_ERR_TIMEOUT, PL_ERR_OVERSUBSCRIBED, PL_ERR_INVALID_SCHEDULE, PL_ERR_OVERFLOW = range(10)
# dtypes
PL_BF16, PL_F32, PL_I32, PL_U8, PL_F32X2 = range(5)
DTYPE_SIZE = {PL_BF16: 2, PL_F32: 4, PL_I32: 4, PL_U8: 1, PL_F32X2: 8}
# collectives
PL_ALLREDUCE, PL_REDUCE_SCATTER, PL_ALLGATHER, PL_ALLTOALL, PL_ALLTOALLV, PL_ALLGATHERV, PL_REDUCE_SCATTERV, \
    PL_BROADCAST, PL_REDUCE, PL_SCATTER, PL_GATHER = range(11)
# algorithms
PL_ALGO_RING, PL_ALGO_TREE, PL_ALGO_DIRECT, PL_ALGO_ONESHOT, PL_ALGO_DIRECT_FUSED, PL_ALGO_AUTO = range(6)
# op kinds / buffer kinds / datapaths
PL_OP_COPY, PL_OP_REDUCE, PL_OP_COPY_REDUCE = range(3)
PL_BUF_IN, PL_BUF_OUT, PL_BUF_SCRATCH = range(3)
PL_DP_AUTO, PL_DP_LDST, PL_DP_TMA, PL_DP_PACKET = range(4)
PL_OPT_SKIP_VALIDATE = 1
PL_OPT_NO_L2_HINTS = 2
PL_OPT_STAGED = 4
PL_OPT_TRACE = 8
PL_OPT_OVERLAP_LAUNCH = 16
PL_OPT_STAGE_AHEAD = 32
PL_OPT_INPUTS_LAST_USE = 64
PL_HOOK_RESIDUAL = 1
PL_HOOK_F32_OUT = 2


class PurlinError(RuntimeError):
    def __init__(self, status, where):
        self.status = status
        super().__init__(f"{where}: {status_string(status)} (status {status})")


class pl_sched_opts_t(C.Structure):
    _fields_ = [("struct_size", C.c_uint32), ("n_ctas", C.c_int32), ("threads", C.c_int32),
                ("datapath", C.c_int32), ("stages", C.c_int32), ("stage_bytes", C.c_uint32),
                ("slice_bytes", C.c_uint32), ("timeout_ns", C.c_uint64), ("flags", C.c_uint32),
                ("staging_bytes", C.c_uint64), ("out_scale", C.c_float), ("hook", C.c_uint32),
                ("idle_sm_first", C.c_int32), ("idle_sm_count", C.c_int32)]


class pl_ref_t(C.Structure):
    _fields_ = [("rank", C.c_int32), ("buf", C.c_int32), ("dtype", C.c_int32), ("pad_", C.c_int32),
                ("offset", C.c_uint64)]


class pl_op_t(C.Structure):
    _fields_ = [("kind", C.c_int32), ("exec_rank", C.c_int32), ("queue", C.c_int32), ("topo", C.c_int32),
                ("layer", C.c_int32), ("n_src", C.c_int32), ("n_wait", C.c_int32), ("signal_flag", C.c_int32),
                ("signal_flag2", C.c_int32), ("dst_bcast", C.c_int32), ("count", C.c_uint64),
                ("dst", pl_ref_t), ("src", pl_ref_t * PL_MAX_SRC),
                ("wait_flag", C.c_int32 * PL_MAX_WAITS), ("wait_need", C.c_uint32 * PL_MAX_WAITS)]


class pl_sched_info_t(C.Structure):
    _fields_ = [("n_ops", C.c_uint64), ("n_queues", C.c_uint64), ("n_flags", C.c_uint64),
                ("n_waits", C.c_uint64), ("n_layers", C.c_uint64),
                ("bytes_read", C.c_uint64), ("bytes_written", C.c_uint64), ("message_bytes", C.c_uint64),
                ("scratch_bytes", C.c_uint64),
                ("in_bytes", C.c_uint64 * PL_MAX_RANKS), ("out_bytes", C.c_uint64 * PL_MAX_RANKS),
                ("grid", C.c_int32), ("threads", C.c_int32), ("smem_bytes", C.c_int32),
                ("datapath", C.c_int32), ("stages", C.c_int32),
                ("stage_bytes", C.c_uint32), ("slice_bytes", C.c_uint32),
                ("aux_bytes", C.c_uint64 * PL_MAX_RANKS), ("out_dtype", C.c_int32), ("hook", C.c_uint32),
                ("hbm_bytes", C.c_uint64), ("idle_sm_first", C.c_int32), ("idle_sm_count", C.c_int32)]


class pl_bufs_t(C.Structure):
    _fields_ = [("in_", C.c_void_p * PL_MAX_RANKS), ("out", C.c_void_p * PL_MAX_RANKS),
                ("in_bytes", C.c_size_t * PL_MAX_RANKS), ("out_bytes", C.c_size_t * PL_MAX_RANKS),
                ("aux", C.c_void_p * PL_MAX_RANKS), ("aux_bytes", C.c_size_t * PL_MAX_RANKS)]


class pl_devstatus_t(C.Structure):
    _fields_ = [("code", C.c_int32), ("queue", C.c_int32), ("op", C.c_int32), ("flag", C.c_int32),
                ("expected", C.c_uint64), ("observed", C.c_uint64)]


EXPORTS = [
    "pl_comm_create", "pl_comm_create_planner", "pl_comm_destroy", "pl_comm_status", "pl_comm_reset",
    "pl_comm_last_error", "pl_probe_hbm",
    "pl_schedule_build", "pl_schedule_build_v", "pl_schedule_build_layers", "pl_schedule_build_rooted", "pl_schedule_info",
    "pl_schedule_dump", "pl_schedule_validate", "pl_schedule_debug_break_wait", "pl_schedule_debug_drop_wait",
    "pl_schedule_trace_read", "pl_schedule_destroy",
    "pl_execute", "pl_execute_host", "pl_execute_host_async", "pl_comm_host_fence", "pl_comm_host_sync", "pl_comm_host_stats", "pl_comm_tune",
    "pl_moe_plan_create", "pl_moe_plan_destroy", "pl_moe_dispatch", "pl_moe_combine", "pl_moe_plan_read",
    "pl_moe_dispatch_dedup", "pl_moe_combine_dedup", "pl_moe_plan_read_dedup", "pl_moe_combine_logits",
    "pl_status_string", "pl_launch_count", "pl_reduce_scatter_ring_static",
    "pl_reduce_scatter_ring_static_debug_timeout",
]

_lib = None


def lib_path() -> str:
    return _build.LIB


def load():
    """Load libpurlin.so (building it in-tree first if it is missing or stale)."""
    global _lib
    if _lib is not None:
        return _lib
    path = _build.LIB
    if _build.needs_build():
        _build.build()
    if not os.path.exists(path):
        raise ImportError(f"{path} is missing: run `python -m paper_2609_36954_b200.build`")
    L = C.CDLL(path)
    vp, i32, u64, sz = C.c_void_p, C.c_int, C.c_uint64, C.c_size_t
    P = C.POINTER
    sig = {
        "pl_comm_create": [i32, i32, P(vp)],
        "pl_comm_create_planner": [i32, i32, P(vp)],
        "pl_comm_destroy": [vp],
        "pl_comm_status": [vp, P(pl_devstatus_t)],
        "pl_comm_reset": [vp, vp],
        "pl_schedule_build": [vp, i32, i32, sz, sz, P(pl_sched_opts_t), P(vp)],
        "pl_schedule_build_v": [vp, i32, i32, P(sz), sz, P(pl_sched_opts_t), P(vp)],
        "pl_schedule_build_layers": [vp, i32, sz, i32, P(pl_sched_opts_t), P(vp)],
        "pl_schedule_build_rooted": [vp, i32, i32, sz, sz, P(pl_sched_opts_t), P(vp)],
        "pl_schedule_info": [vp, P(pl_sched_info_t)],
        "pl_schedule_dump": [vp, P(pl_op_t), sz, P(sz)],
        "pl_schedule_validate": [vp, C.c_char_p, sz],
        "pl_schedule_debug_break_wait": [vp, sz],
        "pl_schedule_debug_drop_wait": [vp, sz],
        "pl_schedule_trace_read": [vp, vp, sz, vp],
        "pl_schedule_destroy": [vp],
        "pl_execute": [vp, P(pl_bufs_t), vp],
        "pl_execute_host": [vp, P(pl_bufs_t), P(pl_bufs_t), vp],
        "pl_execute_host_async": [vp, P(pl_bufs_t), P(pl_bufs_t), vp],
        "pl_comm_host_fence": [vp, vp],
        "pl_comm_host_sync": [vp],
        "pl_comm_host_stats": [vp, P(C.c_uint64), P(C.c_uint64)],
        "pl_comm_tune": [vp, vp, P(C.c_int32), P(C.c_int32), P(C.c_int32)],
        "pl_moe_plan_create": [vp, i32, i32, i32, i32, sz, P(vp)],
        "pl_moe_plan_destroy": [vp],
        "pl_moe_dispatch": [vp, P(vp), P(vp), P(vp), P(vp), vp],
        "pl_moe_combine": [vp, P(vp), P(vp), P(vp), vp],
        "pl_moe_plan_read": [vp, vp, vp, vp, vp],
        "pl_moe_combine_logits": [vp, P(vp), P(vp), P(vp), vp],
        "pl_moe_dispatch_dedup": [vp, P(vp), P(vp), P(vp), P(vp), vp],
        "pl_moe_combine_dedup": [vp, P(vp), P(vp), vp],
        "pl_moe_plan_read_dedup": [vp, vp, vp, vp],
        "pl_reduce_scatter_ring_static": [i32, i32, sz, P(vp), P(vp), vp, vp],
        "pl_reduce_scatter_ring_static_debug_timeout": [i32, i32, sz, P(vp), P(vp), vp, vp, u64],
    }
    for name, args in sig.items():
        fn = getattr(L, name)
        fn.argtypes = args
        fn.restype = C.c_int
    L.pl_status_string.argtypes = [C.c_int]
    L.pl_status_string.restype = C.c_char_p
    L.pl_comm_last_error.argtypes = [vp]
    L.pl_comm_last_error.restype = C.c_char_p
    L.pl_probe_hbm.argtypes = [C.c_int, vp, vp, C.c_size_t, vp, vp]
    L.pl_launch_count.argtypes = []
    L.pl_launch_count.restype = C.c_uint64
    _lib = L
    return L


def status_string(st: int) -> str:
    return load().pl_status_string(int(st)).decode()


def _check(st, where):
    if st != PL_OK:
        raise PurlinError(st, where)


def make_opts(n_ctas=0, threads=0, datapath=PL_DP_AUTO, stages=0, stage_bytes=0, slice_bytes=0,
              timeout_ns=0, flags=0, staging_bytes=0, out_scale=0.0, hook=0, idle_sm_first=0, idle_sm_count=0):
    o = pl_sched_opts_t()
    o.struct_size = C.sizeof(pl_sched_opts_t)
    o.n_ctas, o.threads, o.datapath, o.stages = n_ctas, threads, datapath, stages
    o.stage_bytes, o.slice_bytes, o.timeout_ns, o.flags = stage_bytes, slice_bytes, timeout_ns, flags
    o.staging_bytes = staging_bytes
    o.out_scale = out_scale
    o.hook = hook
    o.idle_sm_first, o.idle_sm_count = idle_sm_first, idle_sm_count
    return o


def make_bufs(ins, outs, in_bytes, out_bytes, aux=None, aux_bytes=None):
    """ins/outs (and aux, for PL_HOOK_RESIDUAL): integer addresses per rank (device or host, as the
    callee expects)."""
    b = pl_bufs_t()
    for r, (a, n) in enumerate(zip(aux or [], aux_bytes or [])):
        b.aux[r] = a
        b.aux_bytes[r] = n
    for r, (a, n) in enumerate(zip(ins, in_bytes)):
        b.in_[r] = a
        b.in_bytes[r] = n
    for r, (a, n) in enumerate(zip(outs, out_bytes)):
        b.out[r] = a
        b.out_bytes[r] = n
    return b


# ---- 1:1 wrappers ---------------------------------------------------------------------
def pl_comm_create(R, dtype):
    h = C.c_void_p()
    _check(load().pl_comm_create(R, dtype, C.byref(h)), "pl_comm_create")
    return h


def pl_comm_create_planner(R, dtype):
    h = C.c_void_p()
    _check(load().pl_comm_create_planner(R, dtype, C.byref(h)), "pl_comm_create_planner")
    return h


def pl_comm_destroy(comm):
    _check(load().pl_comm_destroy(comm), "pl_comm_destroy")


def pl_comm_status(comm):
    s = pl_devstatus_t()
    _check(load().pl_comm_status(comm, C.byref(s)), "pl_comm_status")
    return s


def pl_comm_last_error(comm) -> str:
    return load().pl_comm_last_error(comm).decode()


def pl_probe_hbm(kind: int, src: int, dst: int, nbytes: int, status: int = 0, stream=0) -> None:
    """kind 0 read, 1 write, 2 copy; src / dst / status are device addresses (0 = unused)."""
    _check(load().pl_probe_hbm(kind, src or None, dst or None, nbytes, status or None, stream), "pl_probe_hbm")


def pl_comm_reset(comm, stream=0):
    _check(load().pl_comm_reset(comm, stream), "pl_comm_reset")


def pl_schedule_build(comm, coll, algo, count_per_rank, chunk_bytes, opts=None):
    h = C.c_void_p()
    _check(load().pl_schedule_build(comm, coll, algo, count_per_rank, chunk_bytes,
                                    C.byref(opts) if opts is not None else None, C.byref(h)),
           "pl_schedule_build")
    return h


def pl_schedule_build_v(comm, coll, algo, counts, chunk_bytes, opts=None):
    flat = [int(v) for row in counts for v in (row if hasattr(row, "__len__") else [row])]
    arr = (C.c_size_t * len(flat))(*flat)
    h = C.c_void_p()
    _check(load().pl_schedule_build_v(comm, coll, algo, arr, chunk_bytes,
                                      C.byref(opts) if opts is not None else None, C.byref(h)),
           "pl_schedule_build_v")
    return h


def pl_schedule_build_rooted(comm, coll, root, count_per_rank, chunk_bytes, opts=None):
    h = C.c_void_p()
    _check(load().pl_schedule_build_rooted(comm, coll, root, count_per_rank, chunk_bytes,
                                           C.byref(opts) if opts is not None else None, C.byref(h)),
           "pl_schedule_build_rooted")
    return h


def pl_schedule_build_layers(comm, algo, count_per_rank, n_layers, opts=None):
    h = C.c_void_p()
    _check(load().pl_schedule_build_layers(comm, algo, count_per_rank, n_layers,
                                           C.byref(opts) if opts is not None else None, C.byref(h)),
           "pl_schedule_build_layers")
    return h


def pl_schedule_info(s):
    info = pl_sched_info_t()
    _check(load().pl_schedule_info(s, C.byref(info)), "pl_schedule_info")
    return info


def pl_schedule_dump(s):
    n = C.c_size_t()
    _check(load().pl_schedule_dump(s, None, 0, C.byref(n)), "pl_schedule_dump")
    ops = (pl_op_t * max(1, n.value))()
    _check(load().pl_schedule_dump(s, ops, n.value, C.byref(n)), "pl_schedule_dump")
    return [ops[i] for i in range(n.value)]


def pl_schedule_validate(s):
    buf = C.create_string_buffer(512)
    st = load().pl_schedule_validate(s, buf, 512)
    return st, buf.value.decode()


def pl_schedule_debug_break_wait(s, op_index):
    _check(load().pl_schedule_debug_break_wait(s, op_index), "pl_schedule_debug_break_wait")


def pl_schedule_trace_read(s, n_ops, stream=0):
    """Returns a numpy uint64 array [n_ops, 2] of (start, end) stamps in ns (see purlin.h)."""
    import numpy as np
    out = np.zeros((n_ops, 2), dtype=np.uint64)
    _check(load().pl_schedule_trace_read(s, out.ctypes.data, out.size, stream), "pl_schedule_trace_read")
    return out


def pl_schedule_debug_drop_wait(s, op_index):
    _check(load().pl_schedule_debug_drop_wait(s, op_index), "pl_schedule_debug_drop_wait")


def pl_schedule_destroy(s):
    _check(load().pl_schedule_destroy(s), "pl_schedule_destroy")


def pl_execute(s, bufs, stream=0):
    _check(load().pl_execute(s, C.byref(bufs), stream), "pl_execute")


def pl_execute_host(s, host_bufs, dev_bufs, stream=0):
    _check(load().pl_execute_host(s, C.byref(host_bufs), C.byref(dev_bufs), stream), "pl_execute_host")


def pl_execute_host_async(s, host_bufs, dev_bufs, stream=0):
    _check(load().pl_execute_host_async(s, C.byref(host_bufs), C.byref(dev_bufs), stream), "pl_execute_host_async")


def pl_comm_host_fence(comm, stream=0):
    _check(load().pl_comm_host_fence(comm, stream), "pl_comm_host_fence")


def pl_comm_tune(comm, stream=0, full=False):
    """Returns the grid chosen for pushed copies on the bulk-copy datapath; with full=True the
    tuple (grid, first idle SM, idle SMs) (idle SMs = 0: a plain launch)."""
    g, f, n = C.c_int32(0), C.c_int32(0), C.c_int32(0)
    _check(load().pl_comm_tune(comm, stream, C.byref(g), C.byref(f), C.byref(n)), "pl_comm_tune")
    return (int(g.value), int(f.value), int(n.value)) if full else int(g.value)


def pl_comm_host_stats(comm):
    """(bytes copied host to device, bytes copied device to host) by the host entry points so far."""
    a, b = C.c_uint64(0), C.c_uint64(0)
    _check(load().pl_comm_host_stats(comm, C.byref(a), C.byref(b)), "pl_comm_host_stats")
    return int(a.value), int(b.value)


def pl_comm_host_sync(comm):
    _check(load().pl_comm_host_sync(comm), "pl_comm_host_sync")


def _ptr_array(addrs):
    return (C.c_void_p * len(addrs))(*[int(a) if a else None for a in addrs])


def pl_moe_plan_create(comm, tokens_per_rank, hidden, n_experts, topk, recv_capacity_rows):
    h = C.c_void_p()
    _check(load().pl_moe_plan_create(comm, tokens_per_rank, hidden, n_experts, topk, recv_capacity_rows,
                                     C.byref(h)), "pl_moe_plan_create")
    return h


def pl_moe_plan_destroy(plan):
    _check(load().pl_moe_plan_destroy(plan), "pl_moe_plan_destroy")


def pl_moe_dispatch(plan, x, topk_idx, recv, recv_meta=None, stream=0):
    meta = _ptr_array(recv_meta) if recv_meta is not None else None
    _check(load().pl_moe_dispatch(plan, _ptr_array(x), _ptr_array(topk_idx), _ptr_array(recv), meta, stream),
           "pl_moe_dispatch")


def pl_moe_combine(plan, y, gates, out, stream=0):
    _check(load().pl_moe_combine(plan, _ptr_array(y), _ptr_array(gates), _ptr_array(out), stream),
           "pl_moe_combine")


def pl_moe_combine_logits(plan, y, logits, out, stream=0):
    _check(load().pl_moe_combine_logits(plan, _ptr_array(y), _ptr_array(logits), _ptr_array(out), stream),
           "pl_moe_combine_logits")


def pl_moe_dispatch_dedup(plan, x, topk_idx, recv, recv_meta=None, stream=0):
    meta = _ptr_array(recv_meta) if recv_meta is not None else None
    _check(load().pl_moe_dispatch_dedup(plan, _ptr_array(x), _ptr_array(topk_idx), _ptr_array(recv), meta, stream),
           "pl_moe_dispatch_dedup")


def pl_moe_combine_dedup(plan, z, out, stream=0):
    _check(load().pl_moe_combine_dedup(plan, _ptr_array(z), _ptr_array(out), stream), "pl_moe_combine_dedup")


def pl_moe_plan_read_dedup(plan, pos=0, counts=0, stream=0):
    return load().pl_moe_plan_read_dedup(plan, pos or None, counts or None, stream)


def pl_moe_plan_read(plan, pos=0, counts=0, expert_counts=0, stream=0):
    """pos / counts / expert_counts: host addresses (e.g. numpy ``arr.ctypes.data``) or 0."""
    return load().pl_moe_plan_read(plan, pos or None, counts or None, expert_counts or None, stream)


def pl_reduce_scatter_ring_static(R, dtype, count_per_rank, ins, outs, status=0, stream=0):
    """Ring reduce-scatter that allocates nothing (see include/purlin.h).  ins / outs are
    device addresses per rank; status an optional device address of an int32.  Returns the
    pl_status_t instead of raising, so that callers can test the size limit."""
    return load().pl_reduce_scatter_ring_static(R, dtype, count_per_rank, _ptr_array(ins), _ptr_array(outs),
                                                status or None, stream)


def pl_reduce_scatter_ring_static_debug_timeout(R, dtype, count_per_rank, ins, outs, status, stream, timeout_ns):
    """Test hook: the same call with waits that can never be met and give up after timeout_ns."""
    return load().pl_reduce_scatter_ring_static_debug_timeout(R, dtype, count_per_rank, _ptr_array(ins), _ptr_array(outs),
                                                              status or None, stream, timeout_ns)


def pl_launch_count() -> int:
    return int(load().pl_launch_count())
