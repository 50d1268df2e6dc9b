"""The L2 eviction hints of the bulk-copy datapath change where bytes wait, never what is computed:
schedules built with PL_OPT_INPUTS_LAST_USE (inputs loaded evict-first) or PL_OPT_NO_L2_HINTS give
the same bits as the default ones, and match the oracle."""
import numpy as np
import pytest

from oracle import oracle
from paper_2609_36954_b200 import binding as B
from paper_2609_36954_b200 import inputs as gen

from gpu_harness import Session, check_float

pytestmark = pytest.mark.gpu

CASES = [("rs_direct", B.PL_REDUCE_SCATTER, B.PL_ALGO_DIRECT, 0), ("ag_direct", B.PL_ALLGATHER, B.PL_ALGO_DIRECT, 0),
         ("a2a", B.PL_ALLTOALL, B.PL_ALGO_DIRECT, 0), ("ar_direct", B.PL_ALLREDUCE, B.PL_ALGO_DIRECT, 0),
         ("ar_fused", B.PL_ALLREDUCE, B.PL_ALGO_DIRECT_FUSED, 0), ("ar_ring", B.PL_ALLREDUCE, B.PL_ALGO_RING, 0),
         ("ar_oneshot", B.PL_ALLREDUCE, B.PL_ALGO_ONESHOT, 0),          # reads its inputs R times: the option is ignored
         ("rs_staged", B.PL_REDUCE_SCATTER, B.PL_ALGO_DIRECT, B.PL_OPT_STAGED)]


@pytest.mark.parametrize("name,coll,algo,extra", CASES)
def test_hinted_schedules_give_the_same_bits(name, coll, algo, extra):
    R = 8
    part = 150 * 1024 + 48                      # several ring slots and a ragged tail per partition
    n = R * part // 2
    count = n // R if coll == B.PL_ALLGATHER else n
    x = gen.rank_inputs(R, count, "bf16", seed=91)
    ses = Session(R, "bf16")
    try:
        outs = {}
        for tag, flags in (("default", 0), ("last_use", B.PL_OPT_INPUTS_LAST_USE), ("none", B.PL_OPT_NO_L2_HINTS),
                           ("both", B.PL_OPT_INPUTS_LAST_USE | B.PL_OPT_NO_L2_HINTS)):
            s = ses.build(coll, algo, count, 32768, datapath=B.PL_DP_TMA, flags=flags | extra)
            outs[tag], info = ses.execute(s, x, repeats=2)
            assert info.datapath == B.PL_DP_TMA
        for tag in ("last_use", "none", "both"):
            for r in range(R):
                assert np.array_equal(outs[tag][r], outs["default"][r]), (tag, r)
        if coll == B.PL_REDUCE_SCATTER:
            ref = oracle.reduce_scatter(x, "bf16")
            for r in range(R):
                check_float(gen.bf16_bits_to_f64(outs["last_use"][r].view(np.uint16)), ref[r], "bf16")
        elif coll == B.PL_ALLREDUCE:
            ref = oracle.allreduce(x, "bf16")
            for r in range(R):
                check_float(gen.bf16_bits_to_f64(outs["last_use"][r].view(np.uint16)), ref[r], "bf16")
        elif coll == B.PL_ALLGATHER:
            ref = oracle.allgather(x)
            for r in range(R):
                assert np.array_equal(outs["last_use"][r].view(np.uint16), ref[r])
    finally:
        ses.close()


def test_last_use_is_accepted_and_ignored_off_the_bulk_copy_datapath():
    R, n = 4, 4 * 4096
    x = gen.rank_inputs(R, n, "i32", seed=5)
    ses = Session(R, "i32")
    try:
        for dp in (B.PL_DP_LDST, B.PL_DP_TMA):
            s = ses.build(B.PL_ALLREDUCE, B.PL_ALGO_RING, n, 4096, datapath=dp, flags=B.PL_OPT_INPUTS_LAST_USE)
            outs, _ = ses.execute(s, x)
            ref = oracle.allreduce(x, "i32")
            for r in range(R):
                assert np.array_equal(outs[r].view(np.int32), ref[r])
    finally:
        ses.close()


def test_comm_tune_picks_a_grid_and_later_builds_use_it():
    """pl_comm_tune measures the all-gather's grid on this GPU; the pick is a multiple of R within
    the resident CTAs, later default builds of the pushed all-gather use it, and it computes the
    same bytes as any other grid."""
    R = 8
    ses = Session(R, "bf16")
    try:
        g = B.pl_comm_tune(ses.comm, 0)
        assert g % R == 0 and 96 <= g <= 148
        n = R * (3 << 20)                      # 6 MiB per contribution: the bulk-copy datapath by default
        x = gen.rank_inputs(R, n // R, "bf16", seed=17)
        s = ses.build(B.PL_ALLGATHER, B.PL_ALGO_DIRECT, n // R, 1 << 20, datapath=B.PL_DP_TMA)
        outs, info = ses.execute(s, x)
        assert info.grid == g
        ref = oracle.allgather(x)
        for r in range(R):
            assert np.array_equal(outs[r].view(np.uint16), ref[r])
        s2 = ses.build(B.PL_ALLGATHER, B.PL_ALGO_DIRECT, n // R, 1 << 20, datapath=B.PL_DP_TMA, n_ctas=104)
        assert B.pl_schedule_info(s2).grid == 104                 # an explicit grid still wins
    finally:
        ses.close()
