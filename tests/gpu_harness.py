"""Helpers for the GPU parity tests: device buffers via torch, calls via the C-ABI binding."""
from __future__ import annotations

import numpy as np
import torch

from paper_2609_36954_b200 import binding as B

DT = {"bf16": B.PL_BF16, "f32": B.PL_F32, "i32": B.PL_I32, "u8": B.PL_U8}


def to_dev(a: np.ndarray) -> torch.Tensor:
    """Byte view of a numpy array on cuda:0 (at least 16 bytes so the pointer is valid)."""
    raw = np.ascontiguousarray(a).view(np.uint8).reshape(-1)
    t = torch.empty(max(16, raw.size), dtype=torch.uint8, device="cuda")
    if raw.size:
        t[: raw.size].copy_(torch.from_numpy(raw.copy()))
    return t


def poison(nbytes: int) -> torch.Tensor:
    return torch.full((max(16, int(nbytes)),), 0xFF, dtype=torch.uint8, device="cuda")


def stream_handle() -> int:
    return torch.cuda.current_stream().cuda_stream


class Session:
    """A communicator plus the schedules built on it; destroys them on close."""

    def __init__(self, R, dtype):
        self.R, self.dtype = R, dtype
        self.comm = B.pl_comm_create(R, DT[dtype])
        self.scheds = []

    def build(self, coll, algo, count, chunk, **kw):
        s = B.pl_schedule_build(self.comm, coll, algo, count, chunk, B.make_opts(**kw) if kw else None)
        self.scheds.append(s)
        return s

    def build_v(self, counts, chunk, coll=B.PL_ALLTOALLV, **kw):
        s = B.pl_schedule_build_v(self.comm, coll, B.PL_ALGO_DIRECT, counts, chunk,
                                  B.make_opts(**kw) if kw else None)
        self.scheds.append(s)
        return s

    def build_layers(self, algo, count, n_layers, **kw):
        s = B.pl_schedule_build_layers(self.comm, algo, count, n_layers, B.make_opts(**kw) if kw else None)
        self.scheds.append(s)
        return s

    def execute(self, s, ins_np, repeats=1, d_ins=None):
        """Run schedule s over numpy inputs; returns (list of uint8 numpy outputs, info)."""
        info = B.pl_schedule_info(s)
        R = self.R
        d_in = d_ins if d_ins is not None else [to_dev(a) for a in ins_np]
        d_out = [poison(info.out_bytes[r]) for r in range(R)]
        bufs = B.make_bufs([t.data_ptr() for t in d_in], [t.data_ptr() for t in d_out],
                           [int(info.in_bytes[r]) for r in range(R)], [int(info.out_bytes[r]) for r in range(R)])
        for _ in range(repeats):
            B.pl_execute(s, bufs, stream_handle())
        torch.cuda.synchronize()
        st = B.pl_comm_status(self.comm)
        assert st.code == B.PL_OK, f"device status {st.code} queue {st.queue} op {st.op} flag {st.flag}"
        outs = [d_out[r][: int(info.out_bytes[r])].cpu().numpy() for r in range(R)]
        return outs, info

    def close(self):
        for s in self.scheds:
            B.pl_schedule_destroy(s)
        self.scheds = []
        B.pl_comm_destroy(self.comm)


def check_float(got_f64, ref_f64, dtype):
    """Spec tolerances against the fp64 oracle."""
    if dtype == "bf16":
        tol = 2.0 ** -7 * np.abs(ref_f64) + 1e-6
    else:
        tol = 1e-6 * np.abs(ref_f64) + 1e-7
    err = np.abs(got_f64 - ref_f64)
    bad = err > tol
    assert not bad.any(), f"{int(bad.sum())} elements out of tolerance, max err/tol {float(np.max(err / tol))}"
    return float(np.max(err / tol)) if err.size else 0.0
