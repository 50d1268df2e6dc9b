"""The L2 eviction hints of the bulk-copy datapath change where bytes wait, never what is computed:
schedules built with PL_OPT_INPUTS_LAST_USE (inputs loaded evict-first) or PL_OPT_NO_L2_HINTS give
the same bits as the default ones, and match the oracle."""
import numpy as np
import pytest
import torch

from oracle import oracle
from paper_2609_36954_b200 import binding as B
from paper_2609_36954_b200 import inputs as gen

from gpu_harness import Session, check_float, poison, stream_handle, to_dev

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


def test_sm_window_launch_matches_the_oracle_and_reports_its_window():
    """One CTA per SM is launched, the SMs of the window sit out, the others claim the queues:
    the bytes are those of a plain launch, whatever window is asked for."""
    R = 8
    sms = torch.cuda.get_device_properties(0).multi_processor_count
    n = R * (3 << 20) + R * 4096 * 3
    x = gen.rank_inputs(R, n // R, "bf16", seed=23)
    ref = oracle.allgather(x)
    ses = Session(R, "bf16")
    try:
        for first, count in ((0, sms - 128), (8, sms - 128), (sms - 36, 36), (64, 12)):
            if count <= 0 or (sms - count) % R:
                continue
            s = ses.build(B.PL_ALLGATHER, B.PL_ALGO_DIRECT, n // R, 1 << 20, datapath=B.PL_DP_TMA, idle_sm_first=first, idle_sm_count=count)
            info = B.pl_schedule_info(s)
            assert (info.grid, info.idle_sm_first, info.idle_sm_count) == (sms - count, first, count)
            for rep in range(3):                       # the claim words must be back at zero after every launch
                outs, _ = ses.execute(s, x)
                for r in range(R):
                    assert np.array_equal(outs[r].view(np.uint16), ref[r]), (first, count, rep, r)
        # a reduce-scatter (no flags either) under a window, against the oracle
        xr = gen.rank_inputs(R, n, "bf16", seed=24)
        s = ses.build(B.PL_REDUCE_SCATTER, B.PL_ALGO_DIRECT, n, 1 << 20, datapath=B.PL_DP_TMA, idle_sm_first=16, idle_sm_count=sms - 128)
        outs, _ = ses.execute(s, xr, repeats=2)
        rref = oracle.reduce_scatter(xr, "bf16")
        for r in range(R):
            check_float(gen.bf16_bits_to_f64(outs[r].view(np.uint16)), rref[r], "bf16")
    finally:
        ses.close()


def test_sm_window_launch_keeps_every_queue_when_the_gpu_is_busy():
    """Other work holds SMs while the window launch starts, so its CTAs do not land one per SM at
    once: CTAs on idle SMs that arrive late must pick up what is left, none may run twice."""
    R = 8
    sms = torch.cuda.get_device_properties(0).multi_processor_count
    n = R * (2 << 20)
    x = gen.rank_inputs(R, n // R, "bf16", seed=29)
    ref = oracle.allgather(x)
    ses = Session(R, "bf16")
    try:
        s = ses.build(B.PL_ALLGATHER, B.PL_ALGO_DIRECT, n // R, 1 << 20, datapath=B.PL_DP_TMA, idle_sm_first=8, idle_sm_count=sms - 128)
        info = B.pl_schedule_info(s)
        d_in = [to_dev(a) for a in x]
        d_out = [poison(info.out_bytes[r]) for r in range(R)]
        bufs = B.make_bufs([t.data_ptr() for t in d_in], [t.data_ptr() for t in d_out],
                           [int(info.in_bytes[r]) for r in range(R)], [int(info.out_bytes[r]) for r in range(R)])
        side = torch.cuda.Stream()
        a = torch.randn(4096, 4096, device="cuda")
        for rep in range(6):
            for t in d_out:
                t.fill_(0x5A)
            torch.cuda.synchronize()
            with torch.cuda.stream(side):               # a few milliseconds of work on every SM
                for _ in range(4):
                    a = torch.tanh(a @ a * 1e-4)
            B.pl_execute(s, bufs, stream_handle())
            B.pl_execute(s, bufs, stream_handle())
            torch.cuda.synchronize()
            assert B.pl_comm_status(ses.comm).code == B.PL_OK
            for r in range(R):
                assert np.array_equal(d_out[r][: int(info.out_bytes[r])].cpu().numpy().view(np.uint16), ref[r]), (rep, r)
    finally:
        ses.close()


def test_sm_window_is_rejected_where_it_does_not_apply():
    R = 8
    sms = torch.cuda.get_device_properties(0).multi_processor_count
    ses = Session(R, "bf16")
    try:
        n = R * (1 << 20)
        with pytest.raises(B.PurlinError) as e:       # a ring all-reduce has flags
            ses.build(B.PL_ALLREDUCE, B.PL_ALGO_RING, n, 1 << 18, datapath=B.PL_DP_TMA, idle_sm_first=0, idle_sm_count=sms - 128)
        assert e.value.status == B.PL_ERR_UNSUPPORTED
        with pytest.raises(B.PurlinError) as e:       # the register datapath has no window launch
            ses.build(B.PL_ALLGATHER, B.PL_ALGO_DIRECT, n // R, 1 << 18, datapath=B.PL_DP_LDST, idle_sm_first=0, idle_sm_count=sms - 128)
        assert e.value.status == B.PL_ERR_UNSUPPORTED
        with pytest.raises(B.PurlinError) as e:       # grid and window must add up to the SM count
            ses.build(B.PL_ALLGATHER, B.PL_ALGO_DIRECT, n // R, 1 << 18, datapath=B.PL_DP_TMA, n_ctas=64, idle_sm_first=0, idle_sm_count=sms - 128)
        assert e.value.status == B.PL_ERR_INVALID_ARG
        with pytest.raises(B.PurlinError) as e:       # the other SMs must be a multiple of R
            ses.build(B.PL_ALLGATHER, B.PL_ALGO_DIRECT, n // R, 1 << 18, datapath=B.PL_DP_TMA, idle_sm_first=0, idle_sm_count=sms - 127)
        assert e.value.status == B.PL_ERR_INVALID_ARG
    finally:
        ses.close()


def test_overlapped_launches_never_use_an_sm_window():
    """The claim words of a window launch serve one launch at a time, so a schedule built for
    overlapped launches is a plain launch whatever the tuner found, an explicit window with it is
    refused, and back-to-back overlapped executes of reduce-scatter and all-gather stay correct."""
    R = 8
    sms = torch.cuda.get_device_properties(0).multi_processor_count
    n = R * (2 << 20)
    ses = Session(R, "bf16")
    try:
        with pytest.raises(B.PurlinError) as e:
            ses.build(B.PL_ALLGATHER, B.PL_ALGO_DIRECT, n // R, 1 << 20, datapath=B.PL_DP_TMA, flags=B.PL_OPT_OVERLAP_LAUNCH,
                      idle_sm_first=8, idle_sm_count=sms - 128)
        assert e.value.status == B.PL_ERR_UNSUPPORTED
        ag = ses.build(B.PL_ALLGATHER, B.PL_ALGO_DIRECT, n // R, 1 << 20, datapath=B.PL_DP_TMA, flags=B.PL_OPT_OVERLAP_LAUNCH)
        assert B.pl_schedule_info(ag).idle_sm_count == 0
        rs = ses.build(B.PL_REDUCE_SCATTER, B.PL_ALGO_DIRECT, n, 1 << 20, datapath=B.PL_DP_TMA, flags=B.PL_OPT_OVERLAP_LAUNCH)
        ag_w = ses.build(B.PL_ALLGATHER, B.PL_ALGO_DIRECT, n // R, 1 << 20, datapath=B.PL_DP_TMA)   # default: a window launch
        x = gen.rank_inputs(R, n, "bf16", seed=31)
        irs, iag = B.pl_schedule_info(rs), B.pl_schedule_info(ag_w)
        d_in = [to_dev(a) for a in x]
        d_mid = [poison(irs.out_bytes[r]) for r in range(R)]
        d_out = [poison(iag.out_bytes[r]) for r in range(R)]
        b_rs = B.make_bufs([t.data_ptr() for t in d_in], [t.data_ptr() for t in d_mid], [int(irs.in_bytes[r]) for r in range(R)], [int(irs.out_bytes[r]) for r in range(R)])
        b_ag = B.make_bufs([t.data_ptr() for t in d_mid], [t.data_ptr() for t in d_out], [int(iag.in_bytes[r]) for r in range(R)], [int(iag.out_bytes[r]) for r in range(R)])
        for _ in range(20):                        # overlapped reduce-scatter in front of a window-launched all-gather
            B.pl_execute(rs, b_rs, stream_handle())
            B.pl_execute(ag_w, b_ag, stream_handle())
        torch.cuda.synchronize()
        assert B.pl_comm_status(ses.comm).code == B.PL_OK
        ref = oracle.allreduce(x, "bf16")
        for r in (0, 5):
            check_float(gen.bf16_bits_to_f64(d_out[r][: int(iag.out_bytes[r])].cpu().numpy().view(np.uint16)), ref[r], "bf16")
    finally:
        ses.close()
