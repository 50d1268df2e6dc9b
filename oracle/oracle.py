"""TEST INFRASTRUCTURE ONLY: ctypes front end of the plain-C collectives oracle.

The arithmetic lives in ``collectives_oracle.c`` (naive fp64 / wrapping-int / byte
loops written from the collective definitions of the paper, Sec. 2 and Sec. 3.1,
and the rank-order sum of Sec. 3.3).  This wrapper only marshals numpy arrays.
Nothing in the product package imports this module; only the tests, the smoke
check and the benchmark's cpu_baseline / reference legs do.
"""
from __future__ import annotations

import ctypes
import os
import subprocess

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "collectives_oracle.c")
_LIB = os.path.join(_HERE, "liboracle.so")

BF16, F32, I32, U8 = 0, 1, 2, 3
_lib = None


def build(force: bool = False) -> str:
    """Compile the C oracle (gcc -O2, OpenMP when available)."""
    if not force and os.path.exists(_LIB) and os.path.getmtime(_LIB) >= os.path.getmtime(_SRC):
        return _LIB
    cmd = ["gcc", "-O2", "-std=c99", "-fPIC", "-shared", "-fopenmp", _SRC, "-o", _LIB, "-lm"]
    try:
        subprocess.run(cmd, check=True, capture_output=True)
    except subprocess.CalledProcessError:
        cmd.remove("-fopenmp")
        subprocess.run(cmd, check=True, capture_output=True)
    return _LIB


def lib():
    global _lib
    if _lib is None:
        _lib = ctypes.CDLL(build())
        _lib.orc_num_threads.restype = ctypes.c_int
    return _lib


def num_threads() -> int:
    return int(lib().orc_num_threads())


def _ptrs(arrs):
    for a in arrs:
        assert a.flags["C_CONTIGUOUS"]
    return (ctypes.c_void_p * len(arrs))(*[a.ctypes.data for a in arrs])


def _check(rc, what):
    if rc != 0:
        raise RuntimeError(f"oracle {what} failed with code {rc}")


def allgather(inputs):
    """inputs[r]: any dtype, m bytes each -> out[r] = concatenation over ranks."""
    R = len(inputs)
    m = inputs[0].nbytes
    outs = [np.empty(R * inputs[0].size, dtype=inputs[0].dtype) for _ in range(R)]
    _check(lib().orc_allgather(R, ctypes.c_size_t(m), _ptrs(inputs), _ptrs(outs)), "allgather")
    return outs


def alltoall(inputs):
    R = len(inputs)
    assert inputs[0].nbytes % R == 0
    m = inputs[0].nbytes // R
    outs = [np.empty_like(inputs[0]) for _ in range(R)]
    _check(lib().orc_alltoall(R, ctypes.c_size_t(m), _ptrs(inputs), _ptrs(outs)), "alltoall")
    return outs


def alltoallv(inputs, counts_elems):
    """counts_elems[p][r] = elements p sends to r (element = inputs dtype)."""
    R = len(inputs)
    C = np.ascontiguousarray(np.asarray(counts_elems, dtype=np.uint64) * np.uint64(inputs[0].itemsize))
    outs = [np.zeros(int(np.asarray(counts_elems)[:, r].sum()), dtype=inputs[0].dtype) for r in range(R)]
    # keep zero-size buffers addressable
    outs_c = [o if o.size else np.zeros(1, dtype=o.dtype) for o in outs]
    ins_c = [a if a.size else np.zeros(1, dtype=a.dtype) for a in inputs]
    _check(lib().orc_alltoallv(R, C.ctypes.data_as(ctypes.c_void_p), _ptrs(ins_c), _ptrs(outs_c)), "alltoallv")
    return [oc[:o.size] for oc, o in zip(outs_c, outs)]


def allgatherv(inputs):
    """inputs[p]: rank p's contribution (sizes may differ, may be empty) -> out[r] = concatenation."""
    R = len(inputs)
    nb = np.array([a.nbytes for a in inputs], dtype=np.uint64)
    total = sum(a.size for a in inputs)
    outs = [np.zeros(max(1, total), dtype=inputs[0].dtype) for _ in range(R)]
    ins_c = [a if a.size else np.zeros(1, dtype=a.dtype) for a in inputs]
    _check(lib().orc_allgatherv(R, nb.ctypes.data_as(ctypes.c_void_p), _ptrs(ins_c), _ptrs(outs)), "allgatherv")
    return [o[:total] for o in outs]


def reduce_scatterv(inputs, sizes, dtype):
    """inputs[p]: T = sum(sizes) elements; returns out[k] of sizes[k] elements (fp64 or int32)."""
    R = len(inputs)
    ne = np.array(sizes, dtype=np.uint64)
    assert inputs[0].size == int(ne.sum())
    if dtype == "i32":
        outs = [np.zeros(max(1, int(k)), dtype=np.int32) for k in sizes]
        _check(lib().orc_reduce_scatterv_i32(R, ne.ctypes.data_as(ctypes.c_void_p), _ptrs(inputs), _ptrs(outs)), "rsv_i32")
    else:
        outs = [np.zeros(max(1, int(k)), dtype=np.float64) for k in sizes]
        _check(lib().orc_reduce_scatterv_f64(R, _dtype_code(inputs[0], dtype), ne.ctypes.data_as(ctypes.c_void_p),
                                             _ptrs(inputs), _ptrs(outs)), "rsv_f64")
    return [o[: int(k)] for o, k in zip(outs, sizes)]


def _dtype_code(a, dtype):
    if dtype == "bf16":
        assert a.dtype == np.uint16
        return BF16
    if dtype == "f32":
        assert a.dtype == np.float32
        return F32
    raise ValueError(dtype)


def reduce_scatter(inputs, dtype):
    """dtype 'bf16' (uint16 bits) / 'f32' -> fp64 outputs; 'i32' -> int32 outputs."""
    R = len(inputs)
    n = inputs[0].size
    assert n % R == 0
    m = n // R
    if dtype == "i32":
        outs = [np.empty(m, dtype=np.int32) for _ in range(R)]
        _check(lib().orc_reduce_scatter_i32(R, ctypes.c_size_t(m), _ptrs(inputs), _ptrs(outs)), "rs_i32")
        return outs
    outs = [np.empty(m, dtype=np.float64) for _ in range(R)]
    _check(lib().orc_reduce_scatter_f64(R, _dtype_code(inputs[0], dtype), ctypes.c_size_t(m),
                                        _ptrs(inputs), _ptrs(outs)), "rs_f64")
    return outs


def allreduce(inputs, dtype):
    R = len(inputs)
    n = inputs[0].size
    if dtype == "i32":
        outs = [np.empty(n, dtype=np.int32) for _ in range(R)]
        _check(lib().orc_allreduce_i32(R, ctypes.c_size_t(n), _ptrs(inputs), _ptrs(outs)), "ar_i32")
        return outs
    outs = [np.empty(n, dtype=np.float64) for _ in range(R)]
    _check(lib().orc_allreduce_f64(R, _dtype_code(inputs[0], dtype), ctypes.c_size_t(n),
                                   _ptrs(inputs), _ptrs(outs)), "ar_f64")
    return outs


# ---- rooted collectives (the paper's Appendix B: Broadcast copies the root's entire input to
# every rank, Scatter gives rank r partition r of it, Gather concatenates the contributions in
# rank order at the root, Reduce combines all contributions at the root; the root takes part
# locally in each).  Written with plain numpy slicing; ranks that receive nothing get None.
def broadcast(inputs, root):
    return [np.array(inputs[root], copy=True) for _ in inputs]


def scatter(inputs, root):
    R = len(inputs)
    src = inputs[root]
    assert src.size % R == 0
    m = src.size // R
    return [np.array(src[r * m:(r + 1) * m], copy=True) for r in range(R)]


def gather(inputs, root):
    R = len(inputs)
    out = [None] * R
    out[root] = np.concatenate([inputs[p] for p in range(R)])
    return out


def reduce(inputs, root, dtype):
    """Sum over ranks in ascending rank order from zero, delivered at the root only
    (fp64 for 'bf16'/'f32' inputs, wrapping int32 for 'i32')."""
    R = len(inputs)
    out = [None] * R
    if dtype == "i32":
        acc = np.zeros(inputs[0].size, dtype=np.uint32)
        for p in range(R):
            acc = acc + inputs[p].view(np.uint32)
        out[root] = acc.view(np.int32)
        return out
    acc = np.zeros(inputs[0].size, dtype=np.float64)
    for p in range(R):
        if dtype == "bf16":
            assert inputs[p].dtype == np.uint16
            f = (inputs[p].astype(np.uint32) << np.uint32(16)).view(np.float32).astype(np.float64)
        else:
            f = inputs[p].astype(np.float64)
        acc = acc + f
    out[root] = acc
    return out


# ---- processing phase (Sec. 3.3: the step between the last addition and the store is
# configurable): out_r[i] = scale * sum_p x_p[i] + aux_r[i], all in fp64 here.  The element type of
# the stored result (bf16, or fp32 when no conversion is asked for) is the caller's business: the
# oracle returns the exact fp64 value either way.
def _to_f64(a, dtype):
    if dtype == "bf16":
        assert a.dtype == np.uint16
        return (a.astype(np.uint32) << np.uint32(16)).view(np.float32).astype(np.float64)
    return a.astype(np.float64)


def processed(sums, dtype, scale=1.0, aux=None):
    """sums[r]: fp64 arrays (an fp64 collective result); aux[r]: element-typed second operands laid
    out like the outputs, or None."""
    out = []
    for r, acc in enumerate(sums):
        v = np.float64(scale) * acc
        if aux is not None:
            v = v + _to_f64(aux[r], dtype)
        out.append(v)
    return out


def allreduce_processed(inputs, dtype, scale=1.0, aux=None):
    return processed(allreduce(inputs, dtype), dtype, scale, aux)


def reduce_scatter_processed(inputs, dtype, scale=1.0, aux=None):
    return processed(reduce_scatter(inputs, dtype), dtype, scale, aux)


def moe_dispatch(x, idx, E, recv_capacity_rows=None):
    """x[p]: [T, W] row arrays (any dtype), idx[p]: int32 [T, K].
    Returns dict(recv, meta, pos, counts, expert_counts); recv[r] has capacity rows,
    of which counts[:, r].sum() are valid."""
    R = len(x)
    T, K = idx[0].shape
    row_bytes = x[0].shape[1] * x[0].itemsize
    cap = recv_capacity_rows if recv_capacity_rows is not None else R * T * K
    recv = [np.zeros((cap, x[0].shape[1]), dtype=x[0].dtype) for _ in range(R)]
    meta = [np.full((cap, 4), -1, dtype=np.int32) for _ in range(R)]
    pos = [np.full((T, K), -1, dtype=np.int32) for _ in range(R)]
    counts = np.zeros((R, R), dtype=np.int64)
    ecounts = np.zeros((R, E), dtype=np.int64)
    rc = lib().orc_moe_dispatch(R, T, E, K, ctypes.c_size_t(row_bytes), ctypes.c_size_t(cap),
                                _ptrs(x), _ptrs(idx), _ptrs(recv), _ptrs(meta), _ptrs(pos),
                                counts.ctypes.data_as(ctypes.c_void_p),
                                ecounts.ctypes.data_as(ctypes.c_void_p))
    _check(rc, "moe_dispatch")
    return dict(recv=recv, meta=meta, pos=pos, counts=counts, expert_counts=ecounts)


def moe_combine(y, idx, pos, gates, E, H):
    """y[r]: uint16 bf16 rows [cap, H]; returns fp64 out[p] of shape [T, H]."""
    R = len(y)
    T, K = idx[0].shape
    outs = [np.empty((T, H), dtype=np.float64) for _ in range(R)]
    for a in y:
        assert a.dtype == np.uint16
    for g in gates:
        assert g.dtype == np.float32
    rc = lib().orc_moe_combine_f64(R, T, H, E, K, _ptrs(y), _ptrs(idx), _ptrs(pos), _ptrs(gates), _ptrs(outs))
    _check(rc, "moe_combine")
    return outs


def moe_dispatch_dedup(x, idx, E, recv_capacity_rows=None):
    """One row per (token, destination rank).  Returns dict(recv, meta, pos [T, R], counts)."""
    R = len(x)
    T, K = idx[0].shape
    row_bytes = x[0].shape[1] * x[0].itemsize
    cap = recv_capacity_rows if recv_capacity_rows is not None else R * T
    recv = [np.zeros((cap, x[0].shape[1]), dtype=x[0].dtype) for _ in range(R)]
    meta = [np.full((cap, 4), -1, dtype=np.int32) for _ in range(R)]
    pos = [np.full((T, R), -1, dtype=np.int32) for _ in range(R)]
    counts = np.zeros((R, R), dtype=np.int64)
    rc = lib().orc_moe_dispatch_dedup(R, T, E, K, ctypes.c_size_t(row_bytes), ctypes.c_size_t(cap),
                                      _ptrs(x), _ptrs(idx), _ptrs(recv), _ptrs(meta), _ptrs(pos),
                                      counts.ctypes.data_as(ctypes.c_void_p))
    _check(rc, "moe_dispatch_dedup")
    return dict(recv=recv, meta=meta, pos=pos, counts=counts)


def moe_combine_dedup(z, pos, H):
    """z[r]: uint16 bf16 rows [cap, H] (one per received row); returns fp64 out[p] [T, H]."""
    R = len(z)
    T = pos[0].shape[0]
    outs = [np.empty((T, H), dtype=np.float64) for _ in range(R)]
    rc = lib().orc_moe_combine_dedup_f64(R, T, H, _ptrs(z), _ptrs(pos), _ptrs(outs))
    _check(rc, "moe_combine_dedup")
    return outs
