"""GPU parity of the packet datapath (Sec. 3.2, "Specializing for latency": 8 B payload + 8 B tag
in one 16-byte store, the consumer polls the packet itself) against the CPU oracle, element by
element, plus its epoch reuse, graph replay, trace and time-out behaviour."""
import numpy as np
import pytest
import torch

from oracle import oracle
from paper_2609_36954_b200 import binding as B
from paper_2609_36954_b200 import inputs as gen

from gpu_harness import DT, Session, check_float, poison, stream_handle, to_dev

pytestmark = pytest.mark.gpu

ES = {"bf16": 2, "f32": 4, "i32": 4}


def layered_inputs(R, n, layers, dtype, seed):
    kind = "f32n" if dtype == "f32" else dtype
    per_layer = [gen.rank_inputs(R, n, kind, seed=seed, stream_base=l * R) for l in range(layers)]
    if dtype == "i32":  # the rank-coded integers are the same for every layer: shift them
        per_layer = [[(a.astype(np.int64) + 7919 * l).astype(np.int32) for a in xs] for l, xs in enumerate(per_layer)]
    return [np.concatenate([per_layer[l][r] for l in range(layers)]) for r in range(R)]


def check_layers(outs, x, R, n, layers, dtype):
    for l in range(layers):
        ref = oracle.allreduce([a[l * n:(l + 1) * n] for a in x], dtype)
        for r in range(R):
            if dtype == "i32":
                assert np.array_equal(outs[r].view(np.int32)[l * n:(l + 1) * n], ref[r])
            elif dtype == "bf16":
                check_float(gen.bf16_bits_to_f64(outs[r].view(np.uint16)[l * n:(l + 1) * n]), ref[r], "bf16")
            else:
                check_float(outs[r].view(np.float32)[l * n:(l + 1) * n].astype(np.float64), ref[r], "f32")


@pytest.mark.parametrize("R,dtype,msg_bytes,n_ctas", [
    (8, "bf16", 16384, 0),       # the decode shape: 8 CTAs per rank, 128 threads
    (8, "bf16", 65536, 0),       # 2 vectors per thread
    (8, "bf16", 4096, 0),
    (8, "f32", 16384, 0),
    (8, "i32", 16384, 32),       # 4 CTAs per rank
    (3, "bf16", 16 * 5, 0),      # 5 vectors: one CTA per rank, ragged against the warp
    (2, "i32", 16, 0),           # a single vector
    (16, "bf16", 8192, 0),       # two batches of sources
    (5, "f32", 128 * 1024, 0),   # the largest message: 4 vectors per thread
    (4, "bf16", 2048, 8),        # 2 CTAs per rank
])
def test_packet_layers_match_the_oracle_over_repeated_executes(R, dtype, msg_bytes, n_ctas):
    layers = 7
    n = msg_bytes // ES[dtype]
    ses = Session(R, dtype)
    try:
        s = ses.build_layers(B.PL_ALGO_ONESHOT, n, layers, datapath=B.PL_DP_PACKET, n_ctas=n_ctas)
        info = B.pl_schedule_info(s)
        assert info.datapath == B.PL_DP_PACKET
        for rep in range(3):  # tags carry on from execute to execute; outputs are poisoned every time
            x = layered_inputs(R, n, layers, dtype, seed=30 + rep)
            outs, _ = ses.execute(s, x)
            check_layers(outs, x, R, n, layers, dtype)
    finally:
        ses.close()


def test_packet_path_and_flag_path_give_the_same_bits():
    """Same arithmetic in the same order (ascending rank, fp32, one conversion) on both latency paths."""
    R, n, layers = 8, 8192, 12
    x = layered_inputs(R, n, layers, "bf16", seed=77)
    ses = Session(R, "bf16")
    try:
        a, _ = ses.execute(ses.build_layers(B.PL_ALGO_ONESHOT, n, layers, datapath=B.PL_DP_PACKET), x)
        b, _ = ses.execute(ses.build_layers(B.PL_ALGO_ONESHOT, n, layers), x)
        for r in range(R):
            assert np.array_equal(a[r], b[r])
    finally:
        ses.close()


def test_packet_output_scale_and_odd_layer_count():
    R, n, layers = 8, 2048, 5   # an odd layer count: the buffer parity of layer 0 alternates between executes
    ses = Session(R, "bf16")
    try:
        s = ses.build_layers(B.PL_ALGO_ONESHOT, n, layers, datapath=B.PL_DP_PACKET, out_scale=1.0 / R)
        for rep in range(4):
            x = layered_inputs(R, n, layers, "bf16", seed=90 + rep)
            outs, _ = ses.execute(s, x)
            for l in range(layers):
                ref = oracle.allreduce([a[l * n:(l + 1) * n] for a in x], "bf16")
                for r in range(R):
                    check_float(gen.bf16_bits_to_f64(outs[r].view(np.uint16)[l * n:(l + 1) * n]), ref[r] / R, "bf16")
    finally:
        ses.close()


def test_packet_schedule_in_a_cuda_graph_and_with_overlapped_launches():
    R, n, layers = 8, 8192, 9
    x = layered_inputs(R, n, layers, "bf16", seed=55)
    ses = Session(R, "bf16")
    try:
        for flags in (0, B.PL_OPT_OVERLAP_LAUNCH):
            s = ses.build_layers(B.PL_ALGO_ONESHOT, n, layers, datapath=B.PL_DP_PACKET, flags=flags)
            info = B.pl_schedule_info(s)
            d_in = [to_dev(a) for a in x]
            d_out = [poison(info.out_bytes[r]) for r in range(R)]
            bufs = B.make_bufs([t.data_ptr() for t in d_in], [t.data_ptr() for t in d_out],
                               [int(info.in_bytes[r]) for r in range(R)], [int(info.out_bytes[r]) for r in range(R)])
            B.pl_execute(s, bufs, stream_handle())
            torch.cuda.synchronize()
            g = torch.cuda.CUDAGraph()
            side = torch.cuda.Stream()
            side.wait_stream(torch.cuda.current_stream())
            with torch.cuda.graph(g, stream=side):
                for _ in range(3):
                    B.pl_execute(s, bufs, torch.cuda.current_stream().cuda_stream)
            for _ in range(3):
                for t in d_out:
                    t.fill_(0xFF)
                g.replay()
                torch.cuda.synchronize()
                assert B.pl_comm_status(ses.comm).code == B.PL_OK
                check_layers([t[: int(info.out_bytes[0])].cpu().numpy() for t in d_out], x, R, n, layers, "bf16")
    finally:
        ses.close()


def test_packet_trace_shows_program_order():
    """In-kernel stamps: an op of layer l+1 saw all its packets only after every op of layer l had
    written its slice and was about to join (a rank publishes only once its output is complete)."""
    R, n, layers = 8, 8192, 10
    x = layered_inputs(R, n, layers, "bf16", seed=3)
    ses = Session(R, "bf16")
    try:
        s = ses.build_layers(B.PL_ALGO_ONESHOT, n, layers, datapath=B.PL_DP_PACKET, flags=B.PL_OPT_TRACE)
        outs, _ = ses.execute(s, x, repeats=2)
        check_layers(outs, x, R, n, layers, "bf16")
        ops = B.pl_schedule_dump(s)
        tr = B.pl_schedule_trace_read(s, len(ops))
        start, end = tr[:, 0].astype(np.int64), tr[:, 1].astype(np.int64)
        signallers = {}
        for o in ops:
            if o.signal_flag >= 0:
                signallers.setdefault(o.signal_flag, []).append(o.topo)
        checked = 0
        for o in ops:
            assert start[o.topo] > 0
            for k in range(o.n_wait):
                for sgn in signallers[o.wait_flag[k]]:
                    assert 0 < end[sgn] <= start[o.topo], (o.topo, sgn)
                    checked += 1
        assert checked == (layers - 1) * (len(ops) // layers) ** 2
    finally:
        ses.close()


def test_packet_timeout_is_reported_and_reset_recovers():
    """Host-made failure: one op's polls expect a tag nobody publishes, 20 ms limit.  The clusters
    must all walk out (no thread may be left at a cluster barrier), the status must name the op,
    and after pl_comm_reset the same communicator runs packet schedules correctly again."""
    R, n, layers = 8, 8192, 6
    x = layered_inputs(R, n, layers, "bf16", seed=12)
    ses = Session(R, "bf16")
    try:
        bad = ses.build_layers(B.PL_ALGO_ONESHOT, n, layers, datapath=B.PL_DP_PACKET, timeout_ns=20_000_000)
        good = ses.build_layers(B.PL_ALGO_ONESHOT, n, layers, datapath=B.PL_DP_PACKET)
        outs, _ = ses.execute(good, x)       # leaves tags in the good schedule's buffers
        ops = B.pl_schedule_dump(bad)
        victim = next(o.topo for o in ops if o.layer == 3 and o.exec_rank == 5)
        B.pl_schedule_debug_break_wait(bad, victim)
        info = B.pl_schedule_info(bad)
        d_in = [to_dev(a) for a in x]
        d_out = [poison(info.out_bytes[r]) for r in range(R)]
        bufs = B.make_bufs([t.data_ptr() for t in d_in], [t.data_ptr() for t in d_out],
                           [int(info.in_bytes[r]) for r in range(R)], [int(info.out_bytes[r]) for r in range(R)])
        B.pl_execute(bad, bufs, stream_handle())
        torch.cuda.synchronize()
        st = B.pl_comm_status(ses.comm)
        assert st.code == B.PL_ERR_TIMEOUT and st.expected > st.observed
        # the record names the broken op, or one of the next layer's ops that starved behind it:
        # those wait for the packets of the victim's rank (the flag field holds the missing rank)
        assert st.op == victim or (ops[st.op].layer == 4 and st.flag == 5), (st.op, st.flag)
        B.pl_comm_reset(ses.comm, stream_handle())
        torch.cuda.synchronize()
        assert B.pl_comm_status(ses.comm).code == B.PL_OK
        for rep in range(2):                  # tags restart at 1: the old packets must not be taken for new ones
            x2 = layered_inputs(R, n, layers, "bf16", seed=13 + rep)
            outs, _ = ses.execute(good, x2)
            check_layers(outs, x2, R, n, layers, "bf16")
    finally:
        ses.close()
