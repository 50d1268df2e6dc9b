"""The allocation-free ring reduce-scatter against the schedule-based one.

Some users of this library cannot allocate device memory where they communicate (a serving
loop that must not hit cudaMalloc's synchronisation, code under a fixed memory plan).  For
them pl_reduce_scatter_ring_static keeps its partial sums in an array built into the library.
This file checks that entry point through the C ABI against the existing ring schedule, on two
calls in a row (the built-in array is shared by all calls and keeps the previous call's
contents), plus its size limit.  It is collected last on purpose.
"""
import numpy as np
import pytest
import torch

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


@pytest.mark.parametrize("R,dtype,part_bytes", [
    (8, "bf16", 64 * 1024 + 48),   # ragged against the slice split
    (4, "f32", 128 * 1024),
    (3, "i32", 16),                # one vector per partition: fewer slices than SMs allow
    (2, "bf16", 4096),             # R = 2: no travelling partial at all
])
def test_static_ring_matches_ring_schedule_twice(R, dtype, part_bytes):
    es = B.DTYPE_SIZE[CODE[dtype]]
    n = R * part_bytes // es
    launches = B.pl_launch_count()
    ses = Session(R, dtype)
    try:
        sched = ses.build(B.PL_REDUCE_SCATTER, B.PL_ALGO_RING, n, 65536)
        for call in range(2):  # the second call finds the first call's partial sums in place
            x = gen.rank_inputs(R, n, "f32n" if dtype == "f32" else dtype, seed=20 + call)
            want, _ = ses.execute(sched, x)
            got = run_static(R, dtype, x)
            for r in range(R):
                if dtype == "i32":
                    assert np.array_equal(got[r].view(np.int32), want[r].view(np.int32))
                elif dtype == "bf16":
                    w = gen.bf16_bits_to_f64(want[r].view(np.uint16))
                    check_float(gen.bf16_bits_to_f64(got[r].view(np.uint16)), w, "bf16")
                else:
                    check_float(got[r].view(np.float32).astype(np.float64),
                                want[r].view(np.float32).astype(np.float64), "f32")
    finally:
        ses.close()
    assert B.pl_launch_count() - launches == 4  # two schedule executes + two static calls


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
