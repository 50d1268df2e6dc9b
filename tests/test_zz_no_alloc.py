"""The allocation-free ring reduce-scatter against the oracle and the schedule-based ring.

Some users of this library cannot allocate device memory where they communicate (a serving
loop that must not hit cudaMalloc's synchronisation, code under a fixed memory plan).  For
them pl_reduce_scatter_ring_static keeps its partial sums in an array built into the library.
This file checks that entry point through the C ABI on several calls in a row with changing
inputs (the built-in array is shared by all calls and keeps the previous call's contents):
against the CPU oracle at the usual tolerances, and byte for byte against the existing ring
schedule, which promises the same arithmetic in the same order.  It also covers the size
limit and the time-out path.  It is collected last on purpose.
"""
import numpy as np
import pytest
import torch

from oracle import oracle
from paper_2609_36954_b200 import binding as B
from paper_2609_36954_b200 import inputs as gen

from gpu_harness import Session, check_float, poison, stream_handle, to_dev

pytestmark = pytest.mark.gpu

CODE = {"bf16": B.PL_BF16, "f32": B.PL_F32, "i32": B.PL_I32}


def run_static(R, dtype, x):
    n = x[0].size
    d_in = [to_dev(a) for a in x]
    d_out = [poison(x[0].nbytes // R) for _ in range(R)]
    d_status = torch.full((4,), 7, dtype=torch.int32, device="cuda")
    st = B.pl_reduce_scatter_ring_static(R, CODE[dtype], n, [t.data_ptr() for t in d_in],
                                         [t.data_ptr() for t in d_out], d_status.data_ptr(), stream_handle())
    assert st == B.PL_OK, B.status_string(st)
    torch.cuda.synchronize()
    assert int(d_status[0].item()) == 0
    return [t[: x[0].nbytes // R].cpu().numpy() for t in d_out]


def make_inputs(R, n, dtype, call):
    if dtype == "i32":  # the rank-coded integers, shifted so that every call sees other values
        return [(a.astype(np.int64) + 1000003 * call).astype(np.int32) for a in gen.rank_inputs(R, n, "i32")]
    return gen.rank_inputs(R, n, "f32n" if dtype == "f32" else dtype, seed=20 + call)


def check_against_oracle(got, x, dtype):
    ref = oracle.reduce_scatter(x, dtype)
    for r in range(len(x)):
        if dtype == "i32":
            assert np.array_equal(got[r].view(np.int32), ref[r])          # integers: bit-exact
        elif dtype == "bf16":
            check_float(gen.bf16_bits_to_f64(got[r].view(np.uint16)), ref[r], "bf16")
        else:
            check_float(got[r].view(np.float32).astype(np.float64), ref[r], "f32")


@pytest.mark.parametrize("R,dtype,part_bytes", [
    (8, "bf16", 64 * 1024 + 48),   # ragged against the slice split
    (4, "f32", 128 * 1024),
    (3, "i32", 16),                # one vector per partition: fewer slices than SMs allow
    (2, "bf16", 4096),             # R = 2: no travelling partial at all
])
def test_static_ring_matches_oracle_and_ring_schedule_three_calls(R, dtype, part_bytes):
    es = B.DTYPE_SIZE[CODE[dtype]]
    n = R * part_bytes // es
    launches = B.pl_launch_count()
    ses = Session(R, dtype)
    try:
        sched = ses.build(B.PL_REDUCE_SCATTER, B.PL_ALGO_RING, n, 65536)
        for call in range(3):  # later calls find the earlier calls' partial sums and marks in place
            x = make_inputs(R, n, dtype, call)
            got = run_static(R, dtype, x)
            check_against_oracle(got, x, dtype)
            want, _ = ses.execute(sched, x)
            for r in range(R):     # same partial types, same order of additions: the same bytes
                assert np.array_equal(got[r], want[r])
    finally:
        ses.close()
    assert B.pl_launch_count() - launches == 6  # three schedule executes + three static calls


def test_static_ring_timeout_is_reported_and_the_next_call_is_clean():
    """Host-made failure: the test hook makes every wait expect a mark nobody publishes, with a
    20 ms limit.  The kernel must set the status word and return; a normal call right after it,
    on the same built-in array, must be correct."""
    R, dtype = 4, "bf16"
    n = R * 32 * 1024
    x = make_inputs(R, n, dtype, 7)
    d_in = [to_dev(a) for a in x]
    d_out = [poison(x[0].nbytes // R) for _ in range(R)]
    d_status = torch.zeros(4, dtype=torch.int32, device="cuda")
    ins, outs = [t.data_ptr() for t in d_in], [t.data_ptr() for t in d_out]
    st = B.pl_reduce_scatter_ring_static_debug_timeout(R, CODE[dtype], n, ins, outs, d_status.data_ptr(),
                                                       stream_handle(), 20_000_000)
    assert st == B.PL_OK
    torch.cuda.synchronize()
    assert int(d_status[0].item()) == B.PL_ERR_TIMEOUT
    assert B.pl_reduce_scatter_ring_static_debug_timeout(R, CODE[dtype], n, ins, outs, 0, stream_handle(), 0) \
        == B.PL_ERR_INVALID_ARG
    for call in (8, 9):
        x = make_inputs(R, n, dtype, call)
        check_against_oracle(run_static(R, dtype, x), x, dtype)


def test_static_ring_rejects_what_does_not_fit_and_bad_arguments():
    R = 8
    # 8 * 6 * part * 4 bytes > 32 MiB  <=>  part > 174762 bf16 elements
    n_big = R * 262144
    d = [poison(n_big * 2) for _ in range(R)]
    o = [poison(n_big * 2 // R) for _ in range(R)]
    ins, outs = [t.data_ptr() for t in d], [t.data_ptr() for t in o]
    assert B.pl_reduce_scatter_ring_static(R, B.PL_BF16, n_big, ins, outs) == B.PL_ERR_OVERFLOW
    n_ok = R * 131072
    assert B.pl_reduce_scatter_ring_static(R, B.PL_BF16, n_ok, ins, outs, 0, stream_handle()) == B.PL_OK
    torch.cuda.synchronize()
    assert B.pl_reduce_scatter_ring_static(R, B.PL_U8, n_ok, ins, outs) == B.PL_ERR_UNSUPPORTED
    assert B.pl_reduce_scatter_ring_static(R, B.PL_BF16, n_ok + 8, ins, outs) == B.PL_ERR_INVALID_ARG
    assert B.pl_reduce_scatter_ring_static(R, B.PL_BF16, n_ok, [ins[0] + 2] + ins[1:], outs) == B.PL_ERR_ALIGNMENT
    assert B.pl_reduce_scatter_ring_static(1, B.PL_BF16, n_ok, ins, outs) == B.PL_ERR_INVALID_ARG
