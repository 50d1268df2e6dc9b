"""Property test of the host orchestrator: random communicator sizes, message sizes, chunk and
slice sizes, CTA counts and algorithms; every schedule must validate, replay to the oracle's
result under a random interleaving, and report byte counts that match its own op list."""
import numpy as np
from hypothesis import HealthCheck, given, settings
from hypothesis import strategies as st

from oracle import oracle
from paper_2609_36954_b200 import binding as B
from paper_2609_36954_b200 import inputs as gen

from sched_interp import run as interp_run
from test_orchestrator import DT, compare_reduce

ALGOS = {
    B.PL_ALLREDUCE: [B.PL_ALGO_RING, B.PL_ALGO_TREE, B.PL_ALGO_DIRECT, B.PL_ALGO_ONESHOT, B.PL_ALGO_DIRECT_FUSED],
    B.PL_REDUCE_SCATTER: [B.PL_ALGO_RING, B.PL_ALGO_DIRECT],
    B.PL_ALLGATHER: [B.PL_ALGO_RING, B.PL_ALGO_DIRECT],
    B.PL_ALLTOALL: [B.PL_ALGO_DIRECT],
}


@settings(max_examples=150, deadline=None, suppress_health_check=[HealthCheck.too_slow])
@given(R=st.integers(2, 9), vecs=st.integers(1, 40), chunk_vecs=st.integers(1, 12),
       slice_vecs=st.integers(0, 6), queues=st.integers(1, 5), dtype=st.sampled_from(["i32", "bf16", "f32"]),
       coll=st.sampled_from([B.PL_ALLREDUCE, B.PL_REDUCE_SCATTER, B.PL_ALLGATHER, B.PL_ALLTOALL]),
       algo_i=st.integers(0, 4), staged=st.booleans(), dp=st.sampled_from([B.PL_DP_LDST, B.PL_DP_TMA]),
       seed=st.integers(0, 1000))
def test_random_schedules_validate_and_replay(R, vecs, chunk_vecs, slice_vecs, queues, dtype, coll, algo_i, staged, dp, seed):
    es = B.DTYPE_SIZE[DT[dtype]]
    algos = ALGOS[coll]
    algo = algos[algo_i % len(algos)]
    if staged and algo != B.PL_ALGO_DIRECT:
        staged = False
    n = R * vecs * (16 // es)                                    # elements per rank (vecs vectors per partition)
    count = n // R if coll == B.PL_ALLGATHER else n
    comm = B.pl_comm_create_planner(R, DT[dtype])
    try:
        opts = B.make_opts(n_ctas=queues * R, slice_bytes=16 * slice_vecs, datapath=dp,
                           flags=B.PL_OPT_STAGED if staged else 0,
                           staging_bytes=(R if coll != B.PL_ALLGATHER else 1) * 16 * chunk_vecs * 2 if staged else 0)
        s = B.pl_schedule_build(comm, coll, algo, count, 16 * chunk_vecs, opts)
        st_, msg = B.pl_schedule_validate(s)
        assert st_ == B.PL_OK, msg
        info = B.pl_schedule_info(s)
        ops = B.pl_schedule_dump(s)
        assert len(ops) == info.n_ops and info.n_queues == queues * R
        read = sum(o.count * B.DTYPE_SIZE[o.src[k].dtype] for o in ops for k in range(o.n_src))
        written = sum(o.count * B.DTYPE_SIZE[o.dst.dtype] * (R if o.dst_bcast else 1) for o in ops)
        assert (read, written) == (info.bytes_read, info.bytes_written)
        assert all(0 <= o.queue < queues * R and o.queue % R == o.exec_rank for o in ops)
        x = gen.rank_inputs(R, n, dtype, seed=seed)
        if coll == B.PL_ALLGATHER:
            x = [a[:count].copy() for a in x]
        outs = interp_run(ops, info, R, x, seed=seed)
        if coll == B.PL_ALLREDUCE:
            compare_reduce(outs, oracle.allreduce(x, dtype), dtype)
        elif coll == B.PL_REDUCE_SCATTER:
            compare_reduce(outs, oracle.reduce_scatter(x, dtype), dtype)
        else:
            ref = oracle.allgather(x) if coll == B.PL_ALLGATHER else oracle.alltoall(x)
            for r in range(R):
                assert np.array_equal(outs[r], ref[r].view(np.uint8))
        B.pl_schedule_destroy(s)
    finally:
        B.pl_comm_destroy(comm)
