"""GPU parity: the CUDA path (through the C-ABI) against the CPU oracle, element by element."""
import numpy as np
import pytest

from oracle import oracle
from paper_2609_36954_b200 import binding as B
from paper_2609_36954_b200 import inputs as gen

from gpu_harness import DT, Session, check_float, to_dev

pytestmark = pytest.mark.gpu

ALL_AR = [B.PL_ALGO_RING, B.PL_ALGO_TREE, B.PL_ALGO_DIRECT, B.PL_ALGO_ONESHOT, B.PL_ALGO_DIRECT_FUSED]
ALGO_NAME = {B.PL_ALGO_RING: "ring", B.PL_ALGO_TREE: "tree", B.PL_ALGO_DIRECT: "direct",
             B.PL_ALGO_ONESHOT: "oneshot", B.PL_ALGO_DIRECT_FUSED: "fused"}


def as_f64(out_u8, dtype):
    if dtype == "bf16":
        return gen.bf16_bits_to_f64(out_u8.view(np.uint16))
    return out_u8.view(np.float32).astype(np.float64)


def compare_reduce(outs, ref, dtype):
    worst = 0.0
    for r, o in enumerate(outs):
        if dtype == "i32":
            assert np.array_equal(o.view(np.int32), ref[r]), f"rank {r} differs"
        else:
            worst = max(worst, check_float(as_f64(o, dtype), ref[r], dtype))
    return worst


# ---- config 1: all-reduce R=4, 262144 fp32 + int32 twin, ring, 64 KiB chunks ------------
@pytest.mark.parametrize("dtype", ["f32", "i32"])
def test_config1_allreduce_ring(dtype):
    R, n = 4, 262144
    x = gen.rank_inputs(R, n, dtype, seed=0)
    ref = oracle.allreduce(x, dtype)
    ses = Session(R, dtype)
    try:
        for slice_bytes in (65536, 16384):
            s = ses.build(B.PL_ALLREDUCE, B.PL_ALGO_RING, n, 65536, slice_bytes=slice_bytes)
            outs, info = ses.execute(s, x, repeats=3)  # repeats exercise epoch reuse of the flags
            compare_reduce(outs, ref, dtype)
            if dtype == "i32":  # closed form: 4 i + 262144 * (0+1+2+3)
                i = np.arange(n, dtype=np.int64)
                assert np.array_equal(outs[2].view(np.int32).astype(np.int64), 4 * i + 1572864)
    finally:
        ses.close()


# ---- every all-reduce algorithm, ragged sizes, several R, every dtype ---------------------
DATAPATHS = [B.PL_DP_LDST, B.PL_DP_TMA]


@pytest.mark.parametrize("dp", DATAPATHS)
@pytest.mark.parametrize("algo", ALL_AR)
@pytest.mark.parametrize("dtype", ["bf16", "f32", "i32"])
@pytest.mark.parametrize("R", [2, 3, 8])
def test_allreduce_all_algorithms(algo, dtype, R, dp):
    es = B.DTYPE_SIZE[{"bf16": B.PL_BF16, "f32": B.PL_F32, "i32": B.PL_I32}[dtype]]
    # partition = 37 KiB + 16 B: not a multiple of the chunk, the slice or the CTA width
    n = R * ((37 * 1024 + 16) // es)
    # fp32 data gets full-mantissa N(0,1) values: single-op reductions use a compensated fp32
    # accumulator and multi-hop ones (ring, tree) carry (sum, correction) pairs, so the fp32
    # tolerance holds for any mantissas, not only for the configuration's 2^-23 grid.
    x = gen.rank_inputs(R, n, "f32n" if dtype == "f32" else dtype, seed=11)
    ref = oracle.allreduce(x, dtype)
    ses = Session(R, dtype)
    try:
        for chunk, sl, stage in [(8192, 4096, 2048), (1 << 20, 16384, 32768)]:
            s = ses.build(B.PL_ALLREDUCE, algo, n, chunk, slice_bytes=sl, datapath=dp, stage_bytes=stage, stages=3)
            outs, _ = ses.execute(s, x, repeats=2)
            compare_reduce(outs, ref, dtype)
    finally:
        ses.close()


def test_allreduce_tiny_and_single_vector():
    for R in (2, 5):
        for dtype in ("bf16", "i32"):
            es = 2 if dtype == "bf16" else 4
            n = R * (16 // es)  # one 16-byte vector per partition
            x = gen.rank_inputs(R, n, dtype, seed=1)
            ref = oracle.allreduce(x, dtype)
            ses = Session(R, dtype)
            try:
                for algo in ALL_AR:
                    for dp in DATAPATHS:
                        s = ses.build(B.PL_ALLREDUCE, algo, n, 16, datapath=dp)
                        outs, _ = ses.execute(s, x)
                        compare_reduce(outs, ref, dtype)
            finally:
                ses.close()


@pytest.mark.parametrize("dp", DATAPATHS)
@pytest.mark.parametrize("algo", [B.PL_ALGO_RING, B.PL_ALGO_DIRECT])
@pytest.mark.parametrize("dtype", ["bf16", "i32", "f32"])
def test_reduce_scatter_and_allgather(algo, dtype, dp):
    R = 8
    es = 2 if dtype == "bf16" else 4
    n = R * (300 * 1024 + 48) // es // 1  # partition 300 KiB + 48 B
    n -= n % (R * 16 // es)
    x = gen.rank_inputs(R, n, "f32n" if dtype == "f32" else dtype, seed=3)
    ses = Session(R, dtype)
    try:
        for chunk in (256 * 1024, 1 << 20):
            s = ses.build(B.PL_REDUCE_SCATTER, algo, n, chunk, datapath=dp)
            outs, _ = ses.execute(s, x, repeats=2)
            compare_reduce(outs, oracle.reduce_scatter(x, dtype), dtype)
            m = n // R
            contrib = [a[:m].copy() for a in x]
            s = ses.build(B.PL_ALLGATHER, algo, m, chunk, datapath=dp)
            outs, _ = ses.execute(s, contrib, repeats=2)
            ref = oracle.allgather(contrib)
            for r in range(R):
                assert np.array_equal(outs[r], ref[r].view(np.uint8))
    finally:
        ses.close()


@pytest.mark.parametrize("dp", DATAPATHS)
def test_alltoall_and_alltoallv_bit_exact(dp):
    R = 8
    ses = Session(R, "u8")
    try:
        m = 100 * 1024 + 16
        x = gen.rank_coded_bytes(R, R * m)
        s = ses.build(B.PL_ALLTOALL, B.PL_ALGO_DIRECT, R * m, 65536, datapath=dp)
        outs, _ = ses.execute(s, x)
        ref = oracle.alltoall(x)
        for r in range(R):
            assert np.array_equal(outs[r], ref[r])
        # the paper's Zipf(0.125) split rotated per rank, T = 1 MiB, plus a matrix with empty segments
        for C in (gen.alltoallv_counts_bytes(1 << 20), None):
            if C is None:
                rng = np.random.default_rng(5)
                C = rng.integers(0, 5000, size=(R, R)) * 16
                C[2, :] = 0
                C[:, 5] = 0
            xs = [gen.rank_coded_bytes(R, max(16, int(C[p].sum())))[p][: int(C[p].sum())] for p in range(R)]
            s = ses.build_v(C.tolist(), 65536, datapath=dp)
            outs, info = ses.execute(s, xs)
            ref = oracle.alltoallv(xs, C)
            for r in range(R):
                assert outs[r].size == int(C[:, r].sum())
                assert np.array_equal(outs[r], ref[r])
    finally:
        ses.close()


def test_float_special_cases_on_gpu():
    R, n = 8, 8 * 4096
    base = gen.normal_bf16(n, 11, 0)
    ses = Session(R, "bf16")
    try:
        s = ses.build(B.PL_ALLREDUCE, B.PL_ALGO_DIRECT, n, 65536)
        # all ranks equal -> 8x exactly (power of two), bit-exact even in bf16
        outs, _ = ses.execute(s, [base.copy() for _ in range(R)])
        want = gen.f32_to_bf16_bits((gen.bf16_bits_to_f32(base) * 8).astype(np.float32))
        assert np.array_equal(outs[3].view(np.uint16), want)
        # +x / -x pairs cancel to zero
        neg = base ^ np.uint16(0x8000)
        outs, _ = ses.execute(s, [base if p % 2 == 0 else neg for p in range(R)])
        assert np.all(gen.bf16_bits_to_f32(outs[0].view(np.uint16)) == 0.0)
        # one non-zero rank -> copy of it
        zero = np.zeros(n, np.uint16)
        outs, _ = ses.execute(s, [base if p == 6 else zero for p in range(R)])
        assert np.array_equal(outs[1].view(np.uint16), base)
    finally:
        ses.close()


def test_bf16_direct_sum_is_the_correctly_rounded_sum():
    # fp32 accumulation of 8 bf16 values followed by one rounding reproduces
    # bf16_rne(exact sum) on (nearly) every element; report the fraction, require 99.9 %
    R, n = 8, 8 * 65536
    x = gen.rank_inputs(R, n, "bf16", seed=0)
    ref = oracle.allreduce(x, "bf16")
    ses = Session(R, "bf16")
    try:
        s = ses.build(B.PL_ALLREDUCE, B.PL_ALGO_ONESHOT, n, 1 << 20)
        outs, _ = ses.execute(s, x)
        want = gen.f32_to_bf16_bits(ref[0].astype(np.float32))
        frac = float(np.mean(outs[0].view(np.uint16) == want))
        assert frac > 0.999, frac
    finally:
        ses.close()


@pytest.mark.parametrize("dp", DATAPATHS)
def test_run_to_run_determinism(dp):
    R, n = 8, 8 * 40000
    x = gen.rank_inputs(R, n, "bf16", seed=4)
    ses = Session(R, "bf16")
    try:
        for algo in (B.PL_ALGO_RING, B.PL_ALGO_DIRECT):
            s = ses.build(B.PL_ALLREDUCE, algo, n, 32768, datapath=dp)
            a, _ = ses.execute(s, x)
            b, _ = ses.execute(s, x, repeats=3)
            for r in range(R):
                assert np.array_equal(a[r], b[r])
    finally:
        ses.close()


@pytest.mark.parametrize("algo", [B.PL_ALGO_ONESHOT, B.PL_ALGO_DIRECT, B.PL_ALGO_DIRECT_FUSED])
@pytest.mark.parametrize("batch", [1, 8])
def test_layered_decode_allreduce(algo, batch):
    # tensor-parallel decode shape: batch x hidden 8192 bf16, several layers in one launch
    R, hidden, Lyr = 8, 8192, 6
    n = batch * hidden
    x = [np.concatenate([gen.normal_bf16(n, 0, l * R + r) for l in range(Lyr)]) for r in range(R)]
    ses = Session(R, "bf16")
    try:
        s = ses.build_layers(algo, n, Lyr)
        for rep in range(3):  # back-to-back executes with poisoned outputs: epoch reuse
            outs, info = ses.execute(s, x)
            assert info.n_layers == Lyr
            for l in range(Lyr):
                ref = oracle.allreduce([a[l * n:(l + 1) * n] for a in x], "bf16")
                for r in range(R):
                    check_float(as_f64(outs[r], "bf16")[l * n:(l + 1) * n], ref[r], "bf16")
            x = [np.roll(a, 8 * (rep + 1)) for a in x]  # new inputs next time
    finally:
        ses.close()


def test_execute_argument_errors():
    R, n = 4, 4 * 64
    ses = Session(R, "f32")
    try:
        s = ses.build(B.PL_ALLREDUCE, B.PL_ALGO_ONESHOT, n, 1024)
        info = B.pl_schedule_info(s)
        d_in = [to_dev(np.zeros(n, np.float32)) for _ in range(R)]
        d_out = [to_dev(np.zeros(n + 8, np.float32)) for _ in range(R)]
        ib = [int(info.in_bytes[r]) for r in range(R)]
        ob = [int(info.out_bytes[r]) for r in range(R)]

        def status(bufs):
            with pytest.raises(B.PurlinError) as e:
                B.pl_execute(s, bufs)
            return e.value.status
        ins = [t.data_ptr() for t in d_in]
        outs = [t.data_ptr() for t in d_out]
        assert status(B.make_bufs(ins, [o + 4 for o in outs], ib, ob)) == B.PL_ERR_ALIGNMENT
        assert status(B.make_bufs(ins, outs, ib, [b - 16 for b in ob])) == B.PL_ERR_INVALID_ARG
        assert status(B.make_bufs(ins, [ins[0]] + outs[1:], ib, ob)) == B.PL_ERR_INVALID_ARG  # in/out overlap
        assert status(B.make_bufs([0] + ins[1:], outs, ib, ob)) == B.PL_ERR_INVALID_ARG
        with pytest.raises(B.PurlinError) as e:
            ses.build(B.PL_ALLREDUCE, B.PL_ALGO_ONESHOT, n, 1024, n_ctas=1 << 20)
        assert e.value.status == B.PL_ERR_OVERSUBSCRIBED
    finally:
        ses.close()


@pytest.mark.parametrize("dp", DATAPATHS)
def test_bounded_wait_reports_timeout_and_recovers(dp):
    # host-made failure: one wait edge is raised beyond what the schedule will ever signal;
    # with a 20 ms limit the kernel must return, report PL_ERR_TIMEOUT, and the GPU must stay
    # usable: after pl_comm_reset an intact schedule runs and matches the oracle.
    R, n = 4, 4 * 4096
    x = gen.rank_inputs(R, n, "i32")
    ref = oracle.allreduce(x, "i32")
    ses = Session(R, "i32")
    try:
        bad = ses.build(B.PL_ALLREDUCE, B.PL_ALGO_RING, n, 4096, timeout_ns=20_000_000, datapath=dp)
        ops = B.pl_schedule_dump(bad)
        victim = next(o.topo for o in ops if o.n_wait > 0)
        B.pl_schedule_debug_break_wait(bad, victim)
        info = B.pl_schedule_info(bad)
        import torch
        from gpu_harness import poison, stream_handle
        d_in = [to_dev(a) for a in x]
        d_out = [poison(info.out_bytes[r]) for r in range(R)]
        bufs = B.make_bufs([t.data_ptr() for t in d_in], [t.data_ptr() for t in d_out],
                           [int(info.in_bytes[r]) for r in range(R)], [int(info.out_bytes[r]) for r in range(R)])
        B.pl_execute(bad, bufs, stream_handle())
        torch.cuda.synchronize()
        st = B.pl_comm_status(ses.comm)
        assert st.code == B.PL_ERR_TIMEOUT
        assert st.expected > st.observed
        B.pl_comm_reset(ses.comm, stream_handle())
        torch.cuda.synchronize()
        assert B.pl_comm_status(ses.comm).code == B.PL_OK
        good = ses.build(B.PL_ALLREDUCE, B.PL_ALGO_RING, n, 4096, datapath=dp)
        outs, _ = ses.execute(good, x)
        compare_reduce(outs, ref, "i32")
    finally:
        ses.close()


# ---- staged schedules (ordinary application buffers, cyclic staging) -----------------------
@pytest.mark.parametrize("dp", DATAPATHS)
@pytest.mark.parametrize("dtype", ["bf16", "i32"])
def test_staged_direct_collectives(dp, dtype):
    R = 8
    es = 2 if dtype == "bf16" else 4
    part = 300 * 1024 + 48                      # 5 chunks of 64 KiB (last one short)
    n = R * part // es
    x = gen.rank_inputs(R, n, dtype, seed=9)
    ses = Session(R, dtype)
    try:
        for cap_chunks in (2, 1000):            # 2 slots per partition: every slot is reused; 1000: never
            kw = dict(flags=B.PL_OPT_STAGED, staging_bytes=cap_chunks * R * 65536, datapath=dp)
            s = ses.build(B.PL_ALLREDUCE, B.PL_ALGO_DIRECT, n, 65536, **kw)
            outs, info = ses.execute(s, x, repeats=3)
            compare_reduce(outs, oracle.allreduce(x, dtype), dtype)
            if cap_chunks == 2:
                assert info.scratch_bytes == R * (R * 2 + 2) * 65536
            s = ses.build(B.PL_REDUCE_SCATTER, B.PL_ALGO_DIRECT, n, 65536, **kw)
            outs, _ = ses.execute(s, x, repeats=2)
            compare_reduce(outs, oracle.reduce_scatter(x, dtype), dtype)
            s = ses.build(B.PL_ALLTOALL, B.PL_ALGO_DIRECT, n, 65536, **kw)
            outs, _ = ses.execute(s, x, repeats=2)
            ref = oracle.alltoall(x)
            for r in range(R):
                assert np.array_equal(outs[r], ref[r].view(np.uint8))
            contrib = [a[: n // R].copy() for a in x]
            s = ses.build(B.PL_ALLGATHER, B.PL_ALGO_DIRECT, n // R, 65536,
                          flags=B.PL_OPT_STAGED, staging_bytes=cap_chunks * 65536, datapath=dp)
            outs, _ = ses.execute(s, contrib, repeats=2)
            ref = oracle.allgather(contrib)
            for r in range(R):
                assert np.array_equal(outs[r], ref[r].view(np.uint8))
    finally:
        ses.close()


# ---- V variants with the paper's Zipf(0.125) split ------------------------------------------
@pytest.mark.parametrize("dp", DATAPATHS)
@pytest.mark.parametrize("dtype", ["bf16", "i32"])
def test_allgatherv_and_reduce_scatterv(dp, dtype):
    R = 8
    es = 2 if dtype == "bf16" else 4
    for sizes_b in (gen.zipf_split(4 << 20), np.array([0, 160, 65536 + 16, 0, 48, 300000 // 16 * 16, 16, 1024])):
        sizes = (np.asarray(sizes_b) // es).tolist()
        total = sum(sizes)
        x = gen.rank_inputs(R, total, dtype, seed=13)
        ses = Session(R, dtype)
        try:
            s = ses.build_v(sizes, 65536, coll=B.PL_REDUCE_SCATTERV, datapath=dp)
            outs, info = ses.execute(s, x, repeats=2)
            assert info.message_bytes == total * es
            ref = oracle.reduce_scatterv(x, sizes, dtype)
            for r in range(R):
                assert outs[r].size == sizes[r] * es
                if dtype == "i32":
                    assert np.array_equal(outs[r].view(np.int32), ref[r])
                elif sizes[r]:
                    check_float(as_f64(outs[r], dtype), ref[r], dtype)
            contrib = [x[p][: sizes[p]].copy() for p in range(R)]
            s = ses.build_v(sizes, 65536, coll=B.PL_ALLGATHERV, datapath=dp)
            outs, _ = ses.execute(s, contrib, repeats=2)
            ref = oracle.allgatherv(contrib)
            for r in range(R):
                assert np.array_equal(outs[r], ref[r].view(np.uint8))
        finally:
            ses.close()


# ---- rooted collectives -----------------------------------------------------------------------
@pytest.mark.parametrize("dp", DATAPATHS)
@pytest.mark.parametrize("root", [0, 5])
def test_rooted_collectives(dp, root):
    R = 8
    for dtype in ("bf16", "i32"):
        es = 2 if dtype == "bf16" else 4
        m = (70 * 1024 + 32) // es
        n = R * m
        x = gen.rank_inputs(R, n, dtype, seed=23)
        empty = np.zeros(0, x[0].dtype)
        ses = Session(R, dtype)
        try:
            def run(coll, count, ins):
                s = B.pl_schedule_build_rooted(ses.comm, coll, root, count, 32768, B.make_opts(datapath=dp))
                ses.scheds.append(s)
                return ses.execute(s, ins, repeats=2)
            outs, _ = run(B.PL_BROADCAST, n, [x[r] if r == root else empty for r in range(R)])
            for r in range(R):
                assert np.array_equal(outs[r], x[root].view(np.uint8))
            outs, info = run(B.PL_REDUCE, n, x)
            ref = oracle.reduce(x, root, dtype)[root]
            if dtype == "i32":
                assert np.array_equal(outs[root].view(np.int32), ref)
            else:
                check_float(as_f64(outs[root], dtype), ref, dtype)
            assert all(int(info.out_bytes[r]) == 0 for r in range(R) if r != root)
            outs, _ = run(B.PL_SCATTER, m, [x[r] if r == root else empty for r in range(R)])
            ref = oracle.scatter(x, root)
            for r in range(R):
                assert np.array_equal(outs[r], ref[r].view(np.uint8))
            contrib = [a[:m].copy() for a in x]
            outs, _ = run(B.PL_GATHER, m, contrib)
            assert np.array_equal(outs[root], oracle.gather(contrib, root)[root].view(np.uint8))
        finally:
            ses.close()


# ---- the largest communicator the ABI allows ---------------------------------------------------
@pytest.mark.parametrize("dp", DATAPATHS)
def test_sixteen_ranks(dp):
    R = B.PL_MAX_RANKS
    for dtype in ("bf16", "i32"):
        es = 2 if dtype == "bf16" else 4
        n = R * ((20 * 1024 + 16) // es)
        x = gen.rank_inputs(R, n, dtype, seed=31)
        ref = oracle.allreduce(x, dtype)
        ses = Session(R, dtype)
        try:
            for algo in ALL_AR:
                s = ses.build(B.PL_ALLREDUCE, algo, n, 8192, datapath=dp)
                outs, info = ses.execute(s, x, repeats=2)
                assert info.grid % R == 0
                compare_reduce(outs, ref, dtype)
            s = ses.build(B.PL_ALLTOALL, B.PL_ALGO_DIRECT, n, 8192, datapath=dp)
            outs, _ = ses.execute(s, x)
            a2a = oracle.alltoall(x)
            for r in range(R):
                assert np.array_equal(outs[r], a2a[r].view(np.uint8))
        finally:
            ses.close()


# ---- CUDA-graph replay: the epoch lives on the device, so a captured execute replays correctly ----
@pytest.mark.parametrize("dp", DATAPATHS)
def test_cuda_graph_replay_keeps_results_right(dp):
    import torch
    from gpu_harness import poison
    R, n = 8, 8 * 6000
    x = gen.rank_inputs(R, n, "bf16", seed=41)
    ref = oracle.allreduce(x, "bf16")
    ses = Session(R, "bf16")
    try:
        for algo in (B.PL_ALGO_RING, B.PL_ALGO_DIRECT):
            s = ses.build(B.PL_ALLREDUCE, algo, n, 4096, datapath=dp)
            info = B.pl_schedule_info(s)
            d_in = [to_dev(a) for a in x]
            d_out = [poison(info.out_bytes[r]) for r in range(R)]
            bufs = B.make_bufs([t.data_ptr() for t in d_in], [t.data_ptr() for t in d_out],
                               [int(info.in_bytes[r]) for r in range(R)], [int(info.out_bytes[r]) for r in range(R)])
            B.pl_execute(s, bufs, torch.cuda.current_stream().cuda_stream)   # one plain execute first
            torch.cuda.synchronize()
            g = torch.cuda.CUDAGraph()
            side = torch.cuda.Stream()
            side.wait_stream(torch.cuda.current_stream())
            with torch.cuda.graph(g, stream=side):
                for _ in range(4):                                           # four executes per replay
                    B.pl_execute(s, bufs, torch.cuda.current_stream().cuda_stream)
            for _ in range(3):
                for t in d_out:
                    t.fill_(0xFF)
                g.replay()
                torch.cuda.synchronize()
                assert B.pl_comm_status(ses.comm).code == B.PL_OK
                outs = [d_out[r][: int(info.out_bytes[r])].cpu().numpy() for r in range(R)]
                compare_reduce(outs, ref, "bf16")
            B.pl_execute(s, bufs, torch.cuda.current_stream().cuda_stream)   # and a plain one after the replays
            torch.cuda.synchronize()
            compare_reduce([d_out[r][: int(info.out_bytes[r])].cpu().numpy() for r in range(R)], ref, "bf16")
    finally:
        ses.close()


# ---- processing hook: scaled sums (e.g. an average) ---------------------------------------------
@pytest.mark.parametrize("dp", DATAPATHS)
@pytest.mark.parametrize("dtype", ["bf16", "f32"])
def test_output_scale_hook(dp, dtype):
    R = 8
    es = 2 if dtype == "bf16" else 4
    n = R * ((24 * 1024 + 16) // es)
    x = gen.rank_inputs(R, n, "f32n" if dtype == "f32" else dtype, seed=51)
    scale = np.float32(1.0 / R)
    ses = Session(R, dtype)
    try:
        ref = [a * float(scale) for a in oracle.allreduce(x, dtype)]            # the fp64 sums, scaled
        for algo in ALL_AR:
            s = ses.build(B.PL_ALLREDUCE, algo, n, 8192, datapath=dp, out_scale=float(scale))
            outs, _ = ses.execute(s, x)
            compare_reduce(outs, ref, dtype)
        rs_ref = [a * float(scale) for a in oracle.reduce_scatter(x, dtype)]
        s = ses.build(B.PL_REDUCE_SCATTER, B.PL_ALGO_RING, n, 8192, datapath=dp, out_scale=float(scale))
        outs, _ = ses.execute(s, x)
        compare_reduce(outs, rs_ref, dtype)
        s = B.pl_schedule_build_rooted(ses.comm, B.PL_REDUCE, 2, n, 8192, B.make_opts(datapath=dp, out_scale=float(scale)))
        ses.scheds.append(s)
        outs, _ = ses.execute(s, x)
        check_float(as_f64(outs[2], dtype), oracle.reduce(x, 2, dtype)[2] * float(scale), dtype)
        # copies are untouched by the hook
        s = ses.build(B.PL_ALLTOALL, B.PL_ALGO_DIRECT, n, 8192, datapath=dp, out_scale=float(scale))
        outs, _ = ses.execute(s, x)
        a2a = oracle.alltoall(x)
        for r in range(R):
            assert np.array_equal(outs[r], a2a[r].view(np.uint8))
    finally:
        ses.close()
    si = Session(4, "i32")
    try:
        with pytest.raises(B.PurlinError) as e:
            si.build(B.PL_ALLREDUCE, B.PL_ALGO_DIRECT, 1024, 1024, out_scale=0.5)
        assert e.value.status == B.PL_ERR_UNSUPPORTED
    finally:
        si.close()


# ---- execution trace: on the real device every waiter starts after all of its signallers ended ----
@pytest.mark.parametrize("dp", DATAPATHS)
def test_trace_shows_dependencies_were_respected(dp):
    R = 8
    cases = []
    ses = Session(R, "bf16")
    try:
        n = R * 24 * 1024
        x = gen.rank_inputs(R, n, "bf16", seed=61)
        for algo in (B.PL_ALGO_RING, B.PL_ALGO_TREE, B.PL_ALGO_DIRECT):
            cases.append((ses.build(B.PL_ALLREDUCE, algo, n, 16384, datapath=dp, flags=B.PL_OPT_TRACE), x))
        cases.append((ses.build(B.PL_ALLREDUCE, B.PL_ALGO_DIRECT, n, 16384, datapath=dp,
                                flags=B.PL_OPT_TRACE | B.PL_OPT_STAGED, staging_bytes=2 * R * 16384), x))
        if dp == B.PL_DP_LDST:
            xl = [np.concatenate([gen.normal_bf16(8192, 0, l * R + r) for l in range(10)]) for r in range(R)]
            cases.append((ses.build_layers(B.PL_ALGO_DIRECT_FUSED, 8192, 10, flags=B.PL_OPT_TRACE), xl))
        for s, data in cases:
            ses.execute(s, data, repeats=2)
            ops = B.pl_schedule_dump(s)
            tr = B.pl_schedule_trace_read(s, len(ops))
            start, end = tr[:, 0].astype(np.int64), tr[:, 1].astype(np.int64)
            signallers = {}
            for o in ops:
                for f in (o.signal_flag, o.signal_flag2):
                    if f >= 0:
                        signallers.setdefault(f, []).append(o.topo)
            checked = 0
            for o in ops:
                assert start[o.topo] > 0
                if o.signal_flag >= 0:
                    assert end[o.topo] >= start[o.topo]
                for k in range(o.n_wait):
                    for sgn in signallers[o.wait_flag[k]]:
                        assert 0 < end[sgn] <= start[o.topo], (o.topo, sgn)
                        checked += 1
            assert checked > 0
            # a queue runs its ops in order
            by_q = {}
            for o in sorted(ops, key=lambda o: o.topo):
                by_q.setdefault(o.queue, []).append(start[o.topo])
            assert all(all(b >= a for a, b in zip(v, v[1:])) for v in by_q.values())
        # without the option there is nothing to read
        plain = ses.build(B.PL_ALLREDUCE, B.PL_ALGO_RING, n, 16384, datapath=dp)
        with pytest.raises(B.PurlinError):
            B.pl_schedule_trace_read(plain, 10)
    finally:
        ses.close()


# ---- the two executors run the same arithmetic in the same order: identical bits -------------
def test_register_path_and_bulk_copy_ring_agree_bit_for_bit():
    import torch
    from gpu_harness import poison, stream_handle
    R, n = 8, 8 * 3 * 1024 * 17
    x = gen.rank_inputs(R, n, "bf16", seed=71)
    d_in = [to_dev(a) for a in x]
    ses = Session(R, "bf16")
    try:
        for algo, flags in [(B.PL_ALGO_RING, 0), (B.PL_ALGO_TREE, 0), (B.PL_ALGO_DIRECT, 0), (B.PL_ALGO_DIRECT_FUSED, 0),
                            (B.PL_ALGO_DIRECT, B.PL_OPT_STAGED)]:
            ref = None
            for dp, n_ctas, sl in [(B.PL_DP_LDST, 0, 0), (B.PL_DP_TMA, 0, 0), (B.PL_DP_TMA, 4 * R, 4096), (B.PL_DP_LDST, 9 * R, 8192)]:
                s = ses.build(B.PL_ALLREDUCE, algo, n, 12288, datapath=dp, n_ctas=n_ctas, slice_bytes=sl, flags=flags,
                              staging_bytes=3 * R * 12288 if flags else 0)
                info = B.pl_schedule_info(s)
                d_out = [poison(info.out_bytes[r]) for r in range(R)]
                bufs = B.make_bufs([t.data_ptr() for t in d_in], [t.data_ptr() for t in d_out],
                                   [int(info.in_bytes[r]) for r in range(R)], [int(info.out_bytes[r]) for r in range(R)])
                for _ in range(20):
                    B.pl_execute(s, bufs, stream_handle())
                torch.cuda.synchronize()
                assert B.pl_comm_status(ses.comm).code == B.PL_OK
                out0 = d_out[0][: n * 2].clone()
                assert all(torch.equal(d_out[r][: n * 2], out0) for r in range(1, R))
                if ref is None:
                    ref = out0
                else:
                    assert torch.equal(ref, out0), (algo, dp, n_ctas, sl)
    finally:
        ses.close()


# ---- overlapped launches (programmatic stream serialization) ----------------------------------
@pytest.mark.parametrize("dp", DATAPATHS)
def test_overlapped_launches_keep_stream_order(dp):
    """With PL_OPT_OVERLAP_LAUNCH a kernel's CTAs may start while its predecessor drains; the
    data must still see stream order.  A chain x -> y -> z of two all-reduces where the second
    reads what the first wrote, re-run back to back on poisoned buffers (eagerly and inside a
    CUDA graph), must give all-reduce(all-reduce(x)) every time; repeated executes of ONE
    flagged schedule must keep their epochs apart."""
    import torch
    from gpu_harness import poison
    R, n = 8, 8 * 5000
    x = gen.rank_inputs(R, n, "i32", seed=0)
    y_ref = oracle.allreduce(x, "i32")
    z_ref = oracle.allreduce(y_ref, "i32")
    ses = Session(R, "i32")
    try:
        flags = B.PL_OPT_OVERLAP_LAUNCH
        a = ses.build(B.PL_ALLREDUCE, B.PL_ALGO_RING, n, 2048, datapath=dp, flags=flags)
        b = ses.build(B.PL_ALLREDUCE, B.PL_ALGO_DIRECT, n, 4096, datapath=dp, flags=flags)
        nb = n * 4
        d_x = [to_dev(v) for v in x]
        d_y = [poison(nb) for _ in range(R)]
        d_z = [poison(nb) for _ in range(R)]
        bufs_a = B.make_bufs([t.data_ptr() for t in d_x], [t.data_ptr() for t in d_y], [nb] * R, [nb] * R)
        bufs_b = B.make_bufs([t.data_ptr() for t in d_y], [t.data_ptr() for t in d_z], [nb] * R, [nb] * R)

        def chain(h, reps):
            for _ in range(reps):
                B.pl_execute(a, bufs_a, h)
                B.pl_execute(b, bufs_b, h)

        def check():
            torch.cuda.synchronize()
            assert B.pl_comm_status(ses.comm).code == B.PL_OK
            for r in range(R):
                assert np.array_equal(d_y[r].cpu().numpy().view(np.int32), y_ref[r])
                assert np.array_equal(d_z[r].cpu().numpy().view(np.int32), z_ref[r])

        for _ in range(5):
            for t in d_y + d_z:
                t.fill_(0xFF)
            chain(torch.cuda.current_stream().cuda_stream, 6)
            check()
        g = torch.cuda.CUDAGraph()
        side = torch.cuda.Stream()
        side.wait_stream(torch.cuda.current_stream())
        with torch.cuda.graph(g, stream=side):
            chain(torch.cuda.current_stream().cuda_stream, 8)
        for _ in range(3):
            for t in d_y + d_z:
                t.fill_(0xFF)
            g.replay()
            check()
    finally:
        ses.close()


def test_two_schedules_overlap_on_two_streams_when_co_resident():
    """Executes of different schedules may overlap on the GPU when their grids fit together
    (32 + 32 CTAs here): both chains of flag waits make progress and both results are right."""
    import torch
    from gpu_harness import poison
    R, n = 4, 4 * 20000
    x1 = gen.rank_inputs(R, n, "i32", seed=0)
    x2 = [v + 7 for v in x1]
    ref1, ref2 = oracle.allreduce(x1, "i32"), oracle.allreduce(x2, "i32")
    ses = Session(R, "i32")
    try:
        s1 = ses.build(B.PL_ALLREDUCE, B.PL_ALGO_RING, n, 4096, n_ctas=32, datapath=B.PL_DP_LDST)
        s2 = ses.build(B.PL_ALLREDUCE, B.PL_ALGO_TREE, n, 4096, n_ctas=32, datapath=B.PL_DP_LDST)
        nb = n * 4
        d1, d2 = [to_dev(v) for v in x1], [to_dev(v) for v in x2]
        o1, o2 = [poison(nb) for _ in range(R)], [poison(nb) for _ in range(R)]
        b1 = B.make_bufs([t.data_ptr() for t in d1], [t.data_ptr() for t in o1], [nb] * R, [nb] * R)
        b2 = B.make_bufs([t.data_ptr() for t in d2], [t.data_ptr() for t in o2], [nb] * R, [nb] * R)
        st1, st2 = torch.cuda.Stream(), torch.cuda.Stream()
        torch.cuda.synchronize()
        for _ in range(50):
            B.pl_execute(s1, b1, st1.cuda_stream)
            B.pl_execute(s2, b2, st2.cuda_stream)
        torch.cuda.synchronize()
        assert B.pl_comm_status(ses.comm).code == B.PL_OK
        for r in range(R):
            assert np.array_equal(o1[r].cpu().numpy().view(np.int32), ref1[r])
            assert np.array_equal(o2[r].cpu().numpy().view(np.int32), ref2[r])
    finally:
        ses.close()


def test_stream_probe_copies_and_zero_fills():
    """pl_probe_hbm: the copy stream reproduces its source bit for bit, the write stream leaves
    its pattern, the read stream leaves its source alone; no wait gives up; bad sizes are refused."""
    import torch
    n = 32768 * 301  # ragged against the 148-CTA sweep
    src = torch.randint(0, 255, (n,), dtype=torch.uint8, device="cuda")
    keep = src.clone()
    dst = torch.full((n + 32768,), 7, dtype=torch.uint8, device="cuda")
    status = torch.full((1,), -1, dtype=torch.int32, device="cuda")
    h = torch.cuda.current_stream().cuda_stream
    B.pl_probe_hbm(2, src.data_ptr(), dst.data_ptr(), n, status.data_ptr(), h)
    torch.cuda.synchronize()
    assert int(status.item()) == 0 and torch.equal(dst[:n], src) and bool((dst[n:] == 7).all())
    B.pl_probe_hbm(1, 0, dst.data_ptr(), n, status.data_ptr(), h)
    B.pl_probe_hbm(0, src.data_ptr(), 0, n, status.data_ptr(), h)
    torch.cuda.synchronize()
    pattern = torch.from_numpy(((np.arange(8192, dtype=np.uint64) * 2654435761) % (1 << 32)).astype(np.uint32).view(np.int32)).cuda()
    assert int(status.item()) == 0 and bool((dst[:n].view(torch.int32).view(-1, 8192) == pattern).all()) and bool((dst[n:] == 7).all())
    assert torch.equal(src, keep)
    with pytest.raises(B.PurlinError):
        B.pl_probe_hbm(2, src.data_ptr(), dst.data_ptr(), n - 16, 0, h)
    with pytest.raises(B.PurlinError):
        B.pl_probe_hbm(2, 0, dst.data_ptr(), n, 0, h)


@pytest.mark.parametrize("R", [2, 3, 4, 5, 6, 7, 8])
@pytest.mark.parametrize("dtype", ["bf16", "f32", "i32"])
def test_pipelined_reduce_variant_for_every_source_count(R, dtype):
    """The bulk-copy executor's software-pipelined consumers keep 1, 2 or 4 units per thread
    depending on the source count.  Reduce-scatter and the two-shot all-reduce over ops that
    span several ring stages (and a ragged tail) must match the oracle and, bit for bit, the
    register path, for every R up to 8."""
    import torch
    from gpu_harness import stream_handle
    es = B.DTYPE_SIZE[DT[dtype]]
    per_part = (200 * 1024 + 48) // es          # ~4 stages of 48 KiB per op at R = 8, ragged
    n = R * per_part
    x = gen.rank_inputs(R, n, dtype, seed=90 + R)
    ses = Session(R, dtype)
    try:
        for coll in (B.PL_REDUCE_SCATTER, B.PL_ALLREDUCE):
            ref = oracle.reduce_scatter(x, dtype) if coll == B.PL_REDUCE_SCATTER else oracle.allreduce(x, dtype)
            outs = {}
            for dp in (B.PL_DP_TMA, B.PL_DP_LDST):
                s = ses.build(coll, B.PL_ALGO_DIRECT, n, 1 << 20, datapath=dp)
                if dp == B.PL_DP_TMA:
                    assert B.pl_schedule_info(s).threads == 480   # the 12-warp variant was chosen
                outs[dp], _ = ses.execute(s, x, repeats=3)
                compare_reduce(outs[dp], ref, dtype)
            for r in range(R):
                assert np.array_equal(outs[B.PL_DP_TMA][r], outs[B.PL_DP_LDST][r])
    finally:
        ses.close()
