"""The pipelined host entry point (pl_execute_host_async): uploads, schedule and downloads of
consecutive calls overlap on three streams; the results must be those of the plain, fully
stream-ordered entry point and of the oracle, whatever the buffers share."""
import numpy as np
import pytest
import torch

from oracle import oracle
from paper_2609_36954_b200 import binding as B
from paper_2609_36954_b200 import inputs as gen

from gpu_harness import check_float, stream_handle

pytestmark = pytest.mark.gpu

R = 8


def pinned(a):
    return torch.from_numpy(np.ascontiguousarray(a).view(np.int16)).pin_memory()


def make(ins, outs, info):
    return B.make_bufs([t.data_ptr() for t in ins], [t.data_ptr() for t in outs],
                       [int(info.in_bytes[r]) for r in range(R)], [int(info.out_bytes[r]) for r in range(R)])


def test_reduce_scatter_all_gather_steps_chained_through_host_buffers():
    """Several steps in flight: the all-gather's input host buffer is the reduce-scatter's output host
    buffer (an upload that must wait for a download), the device buffers are the same for every
    step (schedules that must wait for downloads), and the inputs change from step to step."""
    n = R * 512 * 1024                                  # 8 MiB per rank: copies of a millisecond
    steps = 5
    comm = B.pl_comm_create(R, B.PL_BF16)
    try:
        rs = B.pl_schedule_build(comm, B.PL_REDUCE_SCATTER, B.PL_ALGO_DIRECT, n, 1 << 20, None)
        ag = B.pl_schedule_build(comm, B.PL_ALLGATHER, B.PL_ALGO_DIRECT, n // R, 1 << 20, None)
        irs, iag = B.pl_schedule_info(rs), B.pl_schedule_info(ag)
        xs = [gen.rank_inputs(R, n, "bf16", seed=100 + k) for k in range(steps)]
        h_in = [[pinned(a) for a in x] for x in xs]
        h_mid = [torch.empty(n // R, dtype=torch.int16).pin_memory() for _ in range(R)]
        h_out = [[torch.empty(n, dtype=torch.int16).pin_memory() for _ in range(R)] for _ in range(steps)]
        d_in = [torch.empty(n, dtype=torch.int16, device="cuda") for _ in range(R)]
        d_mid = [torch.empty(n // R, dtype=torch.int16, device="cuda") for _ in range(R)]
        d_out = [torch.empty(n, dtype=torch.int16, device="cuda") for _ in range(R)]
        b_rs, b_ag = make(d_in, d_mid, irs), make(d_mid, d_out, iag)
        torch.cuda.synchronize()
        for k in range(steps):
            B.pl_execute_host_async(rs, make(h_in[k], h_mid, irs), b_rs, stream_handle())
            B.pl_execute_host_async(ag, make(h_mid, h_out[k], iag), b_ag, stream_handle())
        B.pl_comm_host_sync(comm)
        assert B.pl_comm_status(comm).code == B.PL_OK
        # the library's own count of what it copied: every output is downloaded; the all-gather's
        # input is not uploaded again while the reduce-scatter's download of it is in flight
        h2d, d2h = B.pl_comm_host_stats(comm)
        full_up = steps * (sum(int(irs.in_bytes[r]) for r in range(R)) + sum(int(iag.in_bytes[r]) for r in range(R)))
        assert d2h == steps * (sum(int(irs.out_bytes[r]) for r in range(R)) + sum(int(iag.out_bytes[r]) for r in range(R)))
        assert steps * sum(int(irs.in_bytes[r]) for r in range(R)) <= h2d <= full_up
        for k in range(steps):
            ref = oracle.allreduce(xs[k], "bf16")
            for r in (0, 3, 7):
                check_float(gen.bf16_bits_to_f64(h_out[k][r].numpy().view(np.uint16)), ref[r], "bf16")
        # the plain entry point after pipelined ones, same buffers: ordered behind their downloads
        B.pl_execute_host_async(rs, make(h_in[0], h_mid, irs), b_rs, stream_handle())
        B.pl_execute_host(ag, make(h_mid, h_out[1], iag), b_ag, stream_handle())
        torch.cuda.synchronize()
        ref = oracle.allreduce(xs[0], "bf16")
        check_float(gen.bf16_bits_to_f64(h_out[1][5].numpy().view(np.uint16)), ref[5], "bf16")
        B.pl_schedule_destroy(rs)
        B.pl_schedule_destroy(ag)
    finally:
        B.pl_comm_destroy(comm)


def test_same_schedule_repeated_into_the_same_buffers_and_fence():
    """One schedule, one set of host and device buffers, different inputs per call: every call's
    schedule overwrites device outputs the previous download reads, every download overwrites the
    host outputs of the previous one.  The last call's result must be there behind the fence."""
    n = R * 256 * 1024
    comm = B.pl_comm_create(R, B.PL_I32)
    try:
        s = B.pl_schedule_build(comm, B.PL_ALLREDUCE, B.PL_ALGO_DIRECT_FUSED, n, 1 << 18, None)
        info = B.pl_schedule_info(s)
        calls = 6
        xs = [[((np.arange(n, dtype=np.int64) * (r + 3) + 17 * k) % 1000003).astype(np.int32) for r in range(R)] for k in range(calls)]
        h_in = [[torch.from_numpy(a).pin_memory() for a in x] for x in xs]
        h_out = [torch.empty(n, dtype=torch.int32).pin_memory() for _ in range(R)]
        d_in = [torch.empty(n, dtype=torch.int32, device="cuda") for _ in range(R)]
        d_out = [torch.empty(n, dtype=torch.int32, device="cuda") for _ in range(R)]
        dev = make(d_in, d_out, info)
        torch.cuda.synchronize()
        for k in range(calls):
            B.pl_execute_host_async(s, make(h_in[k], h_out, info), dev, stream_handle())
        B.pl_comm_host_fence(comm, stream_handle())
        torch.cuda.synchronize()
        want = sum(a.astype(np.int64) for a in xs[-1]).astype(np.int32)
        for r in range(R):
            assert np.array_equal(h_out[r].numpy(), want)
        B.pl_schedule_destroy(s)
    finally:
        B.pl_comm_destroy(comm)


def test_async_host_execute_rejects_what_the_plain_one_rejects():
    comm = B.pl_comm_create(4, B.PL_F32)
    try:
        s = B.pl_schedule_build(comm, B.PL_ALLREDUCE, B.PL_ALGO_RING, 4096, 4096, None)
        info = B.pl_schedule_info(s)
        d = [torch.empty(4096, dtype=torch.float32, device="cuda") for _ in range(8)]
        h = [torch.empty(4096, dtype=torch.float32).pin_memory() for _ in range(8)]
        dev = B.make_bufs([t.data_ptr() for t in d[:4]], [t.data_ptr() for t in d[4:]], [int(info.in_bytes[r]) for r in range(4)], [int(info.out_bytes[r]) for r in range(4)])
        short = B.make_bufs([t.data_ptr() for t in h[:4]], [t.data_ptr() for t in h[4:]], [16] * 4, [int(info.out_bytes[r]) for r in range(4)])
        with pytest.raises(B.PurlinError) as e:
            B.pl_execute_host_async(s, short, dev, stream_handle())
        assert e.value.status == B.PL_ERR_INVALID_ARG
        B.pl_comm_host_sync(comm)          # nothing in flight: returns at once
        B.pl_schedule_destroy(s)
    finally:
        B.pl_comm_destroy(comm)
