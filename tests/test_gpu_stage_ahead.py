"""GPU parity of double-buffered staging (Sec. 4.1-4.2: two staging buffers alternated by epoch
parity so that a rank can enter call n+1 while peers still consume call n): several executes issued
back to back with different inputs and poisoned outputs, every result checked against the oracle."""
import numpy as np
import pytest
import torch

from oracle import oracle
from paper_2609_36954_b200 import binding as B
from paper_2609_36954_b200 import inputs as gen

from gpu_harness import DT, Session, check_float, poison, stream_handle, to_dev

pytestmark = pytest.mark.gpu

FLAGS = B.PL_OPT_STAGED | B.PL_OPT_OVERLAP_LAUNCH | B.PL_OPT_STAGE_AHEAD
ORACLE = {B.PL_ALLREDUCE: lambda x, dt: oracle.allreduce(x, dt), B.PL_REDUCE_SCATTER: lambda x, dt: oracle.reduce_scatter(x, dt),
          B.PL_ALLGATHER: lambda x, dt: oracle.allgather(x), B.PL_ALLTOALL: lambda x, dt: oracle.alltoall(x)}


def make_inputs(R, n, dtype, k):
    if dtype == "i32":
        return [(a.astype(np.int64) * (k + 1) + 977 * k).astype(np.int32) for a in gen.rank_inputs(R, n, "i32")]
    return gen.rank_inputs(R, n, dtype, seed=40 + k)


def check(coll, dtype, outs, ref, R):
    for r in range(R):
        if coll in (B.PL_ALLGATHER, B.PL_ALLTOALL) or dtype == "i32":
            assert np.array_equal(outs[r], np.ascontiguousarray(ref[r]).view(np.uint8).reshape(-1)), f"rank {r}"
        else:
            check_float(gen.bf16_bits_to_f64(outs[r].view(np.uint16)), ref[r], "bf16")


@pytest.mark.parametrize("dp", [B.PL_DP_LDST, B.PL_DP_TMA])
@pytest.mark.parametrize("coll", [B.PL_ALLREDUCE, B.PL_REDUCE_SCATTER, B.PL_ALLGATHER, B.PL_ALLTOALL])
@pytest.mark.parametrize("dtype,cap_chunks", [("bf16", 0), ("i32", 3)])
def test_back_to_back_staged_executes_with_two_staging_buffers(dp, coll, dtype, cap_chunks):
    R, calls = 8, 5
    es = B.DTYPE_SIZE[DT[dtype]]
    chunk = 16384
    part = 5 * chunk + 4096 + 16                       # 6 chunks per partition, ragged tail
    n = (part if coll == B.PL_ALLGATHER else R * part) // es
    cap = cap_chunks * chunk * (1 if coll == B.PL_ALLGATHER else R)   # 3 slots for 6 chunks: cyclic reuse
    ses = Session(R, dtype)
    try:
        s = ses.build(coll, B.PL_ALGO_DIRECT, n, chunk, datapath=dp, flags=FLAGS, staging_bytes=cap)
        info = B.pl_schedule_info(s)
        xs = [make_inputs(R, n, dtype, k) for k in range(calls)]
        d_in = [[to_dev(a) for a in x] for x in xs]
        d_out = [[poison(info.out_bytes[r]) for r in range(R)] for _ in range(calls)]
        ib, ob = [int(info.in_bytes[r]) for r in range(R)], [int(info.out_bytes[r]) for r in range(R)]
        for rep in range(2):                           # the second round starts on the other parity (5 calls)
            for k in range(calls):                     # no synchronisation between the launches
                B.pl_execute(s, B.make_bufs([t.data_ptr() for t in d_in[k]], [t.data_ptr() for t in d_out[k]], ib, ob), stream_handle())
            torch.cuda.synchronize()
            st = B.pl_comm_status(ses.comm)
            assert st.code == B.PL_OK, (st.code, st.queue, st.op, st.flag)
            for k in range(calls):
                outs = [d_out[k][r][: ob[r]].cpu().numpy() for r in range(R)]
                check(coll, dtype, outs, ORACLE[coll](xs[k], dtype), R)
                for t in d_out[k]:
                    t.fill_(0xFF)
    finally:
        ses.close()


def test_double_buffered_schedule_in_a_cuda_graph():
    """The launch number lives on the device, so a captured sequence replays with the right parity."""
    R, n = 8, 8 * 24 * 1024
    x = [gen.rank_inputs(R, n, "bf16", seed=50 + k) for k in range(3)]
    ref = [oracle.allreduce(a, "bf16") for a in x]
    ses = Session(R, "bf16")
    try:
        s = ses.build(B.PL_ALLREDUCE, B.PL_ALGO_DIRECT, n, 16384, flags=FLAGS)
        info = B.pl_schedule_info(s)
        ib, ob = [int(info.in_bytes[r]) for r in range(R)], [int(info.out_bytes[r]) for r in range(R)]
        d_in = [[to_dev(a) for a in xk] for xk in x]
        d_out = [[poison(ob[r]) for r in range(R)] for _ in range(3)]
        bufs = [B.make_bufs([t.data_ptr() for t in d_in[k]], [t.data_ptr() for t in d_out[k]], ib, ob) for k in range(3)]
        B.pl_execute(s, bufs[0], stream_handle())      # an odd number of launches before the capture
        torch.cuda.synchronize()
        g = torch.cuda.CUDAGraph()
        side = torch.cuda.Stream()
        side.wait_stream(torch.cuda.current_stream())
        with torch.cuda.graph(g, stream=side):
            for k in range(3):
                B.pl_execute(s, bufs[k], torch.cuda.current_stream().cuda_stream)
        for _ in range(3):
            for k in range(3):
                for t in d_out[k]:
                    t.fill_(0xFF)
            g.replay()
            torch.cuda.synchronize()
            assert B.pl_comm_status(ses.comm).code == B.PL_OK
            for k in range(3):
                for r in range(R):
                    check_float(gen.bf16_bits_to_f64(d_out[k][r][: ob[r]].cpu().numpy().view(np.uint16)), ref[k][r], "bf16")
    finally:
        ses.close()
