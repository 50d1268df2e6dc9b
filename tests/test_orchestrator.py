"""Host orchestrator (planner communicator, no GPU): lowering, validation, error rules, and
replay of the dumped op lists on the CPU against the oracle."""
import numpy as np
import pytest

from oracle import oracle
from paper_2609_36954_b200 import binding as B
from paper_2609_36954_b200 import inputs as gen

from sched_interp import run as interp_run

DT = {"bf16": B.PL_BF16, "f32": B.PL_F32, "i32": B.PL_I32, "u8": B.PL_U8}
NP = {"bf16": np.uint16, "f32": np.float32, "i32": np.int32, "u8": np.uint8}


def check_float(got_f64, ref_f64, dtype):
    if dtype == "bf16":
        tol = 2.0 ** -7 * np.abs(ref_f64) + 1e-6
    else:
        tol = 1e-6 * np.abs(ref_f64) + 1e-7
    err = np.abs(got_f64 - ref_f64)
    assert np.all(err <= tol), f"max err/tol {np.max(err / tol)}"


def compare_reduce(outs_u8, ref, dtype):
    for r, o in enumerate(outs_u8):
        if dtype == "i32":
            assert np.array_equal(o.view(np.int32), ref[r])
        elif dtype == "bf16":
            check_float(gen.bf16_bits_to_f64(o.view(np.uint16)), ref[r], dtype)
        else:
            check_float(o.view(np.float32).astype(np.float64), ref[r], dtype)


class Planner:
    def __init__(self, R, dtype):
        self.R, self.dtype = R, dtype
        self.comm = B.pl_comm_create_planner(R, DT[dtype])
        self.scheds = []

    def build(self, coll, algo, count, chunk, **kw):
        s = B.pl_schedule_build(self.comm, coll, algo, count, chunk, B.make_opts(**kw) if kw else None)
        self.scheds.append(s)
        return s

    def close(self):
        for s in self.scheds:
            B.pl_schedule_destroy(s)
        B.pl_comm_destroy(self.comm)


ALLREDUCE_ALGOS = [B.PL_ALGO_RING, B.PL_ALGO_TREE, B.PL_ALGO_DIRECT, B.PL_ALGO_ONESHOT, B.PL_ALGO_DIRECT_FUSED]


@pytest.mark.parametrize("R", [2, 3, 4, 5, 8])
@pytest.mark.parametrize("algo", ALLREDUCE_ALGOS)
@pytest.mark.parametrize("dtype", ["i32", "bf16", "f32"])
def test_allreduce_schedules_replay_to_oracle(R, algo, dtype):
    es = B.DTYPE_SIZE[DT[dtype]]
    n = R * (16 // es) * 13  # 13 vectors per partition: ragged against every chunk size below
    x = gen.rank_inputs(R, n, dtype, seed=R)
    ref = oracle.allreduce(x, dtype)
    pl = Planner(R, dtype)
    try:
        for chunk, slice_b in [(16, 16), (48, 32), (1 << 20, 64), (64, 0)]:
            s = pl.build(B.PL_ALLREDUCE, algo, n, chunk, slice_bytes=slice_b, n_ctas=3 * R)
            st, msg = B.pl_schedule_validate(s)
            assert st == B.PL_OK, msg
            info = B.pl_schedule_info(s)
            ops = B.pl_schedule_dump(s)
            assert len(ops) == info.n_ops
            for seed in (0, 1):
                outs = interp_run(ops, info, R, x, seed=seed)
                compare_reduce(outs, ref, dtype)
    finally:
        pl.close()


@pytest.mark.parametrize("R", [2, 3, 5, 8])
@pytest.mark.parametrize("algo", [B.PL_ALGO_RING, B.PL_ALGO_DIRECT])
def test_reduce_scatter_and_allgather_replay(R, algo):
    for dtype in ("i32", "bf16"):
        es = B.DTYPE_SIZE[DT[dtype]]
        n = R * (16 // es) * 7
        x = gen.rank_inputs(R, n, dtype, seed=7)
        pl = Planner(R, dtype)
        try:
            s = pl.build(B.PL_REDUCE_SCATTER, algo, n, 48, slice_bytes=32, n_ctas=2 * R)
            info = B.pl_schedule_info(s)
            outs = interp_run(B.pl_schedule_dump(s), info, R, x, seed=3)
            compare_reduce(outs, oracle.reduce_scatter(x, dtype), dtype)
            assert info.message_bytes == n * es
            # all-gather of the same buffers (contribution = n elements)
            s = pl.build(B.PL_ALLGATHER, algo, n, 48, slice_bytes=32, n_ctas=2 * R)
            info = B.pl_schedule_info(s)
            outs = interp_run(B.pl_schedule_dump(s), info, R, x, seed=4)
            ref = oracle.allgather(x)
            for r in range(R):
                assert np.array_equal(outs[r], ref[r].view(np.uint8))
            assert info.message_bytes == n * es * R
        finally:
            pl.close()


@pytest.mark.parametrize("R", [2, 4, 7])
def test_alltoall_and_alltoallv_replay(R):
    pl = Planner(R, "u8")
    try:
        m = 16 * 5
        x = gen.rank_coded_bytes(R, R * m)
        s = pl.build(B.PL_ALLTOALL, B.PL_ALGO_DIRECT, R * m, 32, slice_bytes=16)
        outs = interp_run(B.pl_schedule_dump(s), B.pl_schedule_info(s), R, x)
        ref = oracle.alltoall(x)
        for r in range(R):
            assert np.array_equal(outs[r], ref[r])
        rng = np.random.default_rng(R)
        C = rng.integers(0, 6, size=(R, R)) * 16
        C[0, R - 1] = 0
        xs = [gen.rank_coded_bytes(R, max(16, int(C[p].sum())))[p][: int(C[p].sum())] for p in range(R)]
        s = B.pl_schedule_build_v(pl.comm, B.PL_ALLTOALLV, B.PL_ALGO_DIRECT, C.tolist(), 48, None)
        pl.scheds.append(s)
        info = B.pl_schedule_info(s)
        outs = interp_run(B.pl_schedule_dump(s), info, R, xs)
        ref = oracle.alltoallv(xs, C)
        for r in range(R):
            assert int(info.out_bytes[r]) == int(C[:, r].sum())
            assert np.array_equal(outs[r], ref[r])
    finally:
        pl.close()


@pytest.mark.parametrize("algo", [B.PL_ALGO_ONESHOT, B.PL_ALGO_DIRECT, B.PL_ALGO_DIRECT_FUSED])
def test_layered_allreduce_replay_and_program_order(algo):
    R, n, Lyr = 4, 4 * 8 * 3, 5
    dtype = "bf16"
    pl = Planner(R, dtype)
    try:
        x = [np.concatenate([gen.normal_bf16(n, 0, l * R + r) for l in range(Lyr)]) for r in range(R)]
        s = B.pl_schedule_build_layers(pl.comm, algo, n, Lyr, B.make_opts(slice_bytes=32, n_ctas=2 * R))
        pl.scheds.append(s)
        st, msg = B.pl_schedule_validate(s)
        assert st == B.PL_OK, msg
        info = B.pl_schedule_info(s)
        assert info.n_layers == Lyr
        ops = B.pl_schedule_dump(s)
        outs = interp_run(ops, info, R, x, seed=5)
        for l in range(Lyr):
            xl = [a[l * n:(l + 1) * n] for a in x]
            ref = oracle.allreduce(xl, dtype)
            for r in range(R):
                got = gen.bf16_bits_to_f64(outs[r].view(np.uint16)[l * n:(l + 1) * n])
                check_float(got, ref[r], dtype)
        # program order: an op of layer l+1 that reads rank p's input waits on a flag that is
        # only complete once every op writing out_p in layer l has signalled
        writers = {}
        for o in ops:
            for f in (o.signal_flag, o.signal_flag2):
                if f >= 0:
                    writers.setdefault(f, []).append(o)
        for o in ops:
            if o.layer == 0 or o.kind == B.PL_OP_COPY:
                continue
            waited = {o.wait_flag[k] for k in range(o.n_wait)}
            for k in range(o.n_src):
                p = o.src[k].rank
                prev_writers = [w for w in ops if w.layer == o.layer - 1 and
                                (w.dst_bcast or w.dst.rank == p) and w.dst.buf == B.PL_BUF_OUT]
                assert prev_writers
                for w in prev_writers:
                    assert {w.signal_flag, w.signal_flag2} & waited, "missing cross-layer edge"
    finally:
        pl.close()


@pytest.mark.parametrize("R,units,G", [(4, 24, 0), (8, 64, 8), (3, 5, 0), (2, 16, 2)])
def test_packet_schedule_replay_program_order_and_geometry(R, units, G):
    """The packet datapath's schedule: the op list states the data movement and the ordering rules
    (as logical flags); replayed on the CPU it must give the oracle's all-reduce per layer, every
    cross-layer edge must be there, and op (layer, rank, slice) must sit at the index the kernel
    derives from its block index."""
    dtype, Lyr = "bf16", 4
    n = units * 8
    pl = Planner(R, dtype)
    try:
        x = [np.concatenate([gen.normal_bf16(n, 0, l * R + r) for l in range(Lyr)]) for r in range(R)]
        s = B.pl_schedule_build_layers(pl.comm, B.PL_ALGO_AUTO, n, Lyr, B.make_opts(datapath=B.PL_DP_PACKET, n_ctas=G * R))
        pl.scheds.append(s)
        assert B.pl_schedule_validate(s)[0] == B.PL_OK
        info = B.pl_schedule_info(s)
        assert info.datapath == B.PL_DP_PACKET and info.n_layers == Lyr
        g = int(info.grid) // R
        assert g in (1, 2, 4, 8) and units % g == 0 and (G == 0 or g == G)
        assert info.scratch_bytes == R * 4 * n * 2          # two packet buffers of twice the message per rank
        ops = B.pl_schedule_dump(s)
        assert len(ops) == Lyr * R * g
        for o in ops:
            r, j = o.exec_rank, o.queue // R
            assert o.topo == (o.layer * R + r) * g + j and o.queue % R == r
            assert o.count == n // g and o.dst.offset == (o.layer * n + j * (n // g)) * 2
            assert o.n_wait == (R if o.layer else 0)
        outs = interp_run(ops, info, R, x, seed=9)
        for l in range(Lyr):
            ref = oracle.allreduce([a[l * n:(l + 1) * n] for a in x], dtype)
            for r in range(R):
                check_float(gen.bf16_bits_to_f64(outs[r].view(np.uint16)[l * n:(l + 1) * n]), ref[r], dtype)
        writers = {}
        for o in ops:
            if o.signal_flag >= 0:
                writers.setdefault(o.signal_flag, []).append(o)
        for o in ops:
            if o.layer:
                waited = {o.wait_flag[k] for k in range(o.n_wait)}
                for w in ops:
                    if w.layer == o.layer - 1:
                        assert w.signal_flag in waited
    finally:
        pl.close()


def test_layers_auto_picks_packets_for_tiny_messages_only():
    pl = Planner(8, "bf16")
    try:
        for n, want_dp, want_grid in ((512, B.PL_DP_PACKET, 8), (2048, B.PL_DP_PACKET, 8), (4096, B.PL_DP_LDST, None), (8192, B.PL_DP_LDST, None)):
            s = B.pl_schedule_build_layers(pl.comm, B.PL_ALGO_AUTO, n, 4, None)
            pl.scheds.append(s)
            info = B.pl_schedule_info(s)
            assert info.datapath == want_dp, (n, info.datapath)
            if want_grid:
                assert info.grid == want_grid          # one CTA per rank
        # anything the caller pins keeps the flag path
        s = B.pl_schedule_build_layers(pl.comm, B.PL_ALGO_AUTO, 512, 4, B.make_opts(n_ctas=16))
        pl.scheds.append(s)
        assert B.pl_schedule_info(s).datapath == B.PL_DP_LDST
        s = B.pl_schedule_build_layers(pl.comm, B.PL_ALGO_DIRECT_FUSED, 512, 4, None)
        pl.scheds.append(s)
        assert B.pl_schedule_info(s).datapath == B.PL_DP_LDST
    finally:
        pl.close()


def test_packet_schedule_rejections():
    pl = Planner(4, "bf16")
    try:
        pk = B.make_opts(datapath=B.PL_DP_PACKET)
        for algo in (B.PL_ALGO_DIRECT, B.PL_ALGO_DIRECT_FUSED, B.PL_ALGO_RING):
            with pytest.raises(B.PurlinError) as e:
                B.pl_schedule_build_layers(pl.comm, algo, 1024, 3, pk)
            assert e.value.status == B.PL_ERR_UNSUPPORTED
        with pytest.raises(B.PurlinError) as e:   # not a layered build
            B.pl_schedule_build(pl.comm, B.PL_ALLREDUCE, B.PL_ALGO_ONESHOT, 1024, 1024, pk)
        assert e.value.status == B.PL_ERR_UNSUPPORTED
        with pytest.raises(B.PurlinError) as e:   # 1 MiB per rank: beyond what a CTA's threads can hold
            B.pl_schedule_build_layers(pl.comm, B.PL_ALGO_ONESHOT, 512 * 1024, 2, pk)
        assert e.value.status == B.PL_ERR_UNSUPPORTED
        with pytest.raises(B.PurlinError) as e:   # 3 CTAs per rank
            B.pl_schedule_build_layers(pl.comm, B.PL_ALGO_ONESHOT, 1024, 2, B.make_opts(datapath=B.PL_DP_PACKET, n_ctas=12))
        assert e.value.status == B.PL_ERR_INVALID_ARG
        with pytest.raises(B.PurlinError) as e:   # 24 bytes
            B.pl_schedule_build_layers(pl.comm, B.PL_ALGO_ONESHOT, 12, 2, pk)
        assert e.value.status == B.PL_ERR_INVALID_ARG
    finally:
        pl.close()
    pu = Planner(4, "u8")
    try:
        with pytest.raises(B.PurlinError) as e:
            B.pl_schedule_build_layers(pu.comm, B.PL_ALGO_ONESHOT, 1024, 2, B.make_opts(datapath=B.PL_DP_PACKET))
        assert e.value.status == B.PL_ERR_UNSUPPORTED
    finally:
        pu.close()


@pytest.mark.parametrize("hook", [B.PL_HOOK_RESIDUAL, B.PL_HOOK_F32_OUT, B.PL_HOOK_RESIDUAL | B.PL_HOOK_F32_OUT])
def test_processing_hooks_lowering_and_replay(hook):
    """Schedules with a processing phase: the reduce ops that write output are flagged final, fp32
    output doubles the output bytes and offsets of a bf16 schedule, the second operand is sized like
    the element-typed output; replayed on the CPU the schedule gives scale * sum + aux."""
    R, dtype = 4, "bf16"
    n = R * 8 * 5
    scale = 0.25
    x = [gen.normal_bf16(n, 0, r) for r in range(R)]
    pl = Planner(R, dtype)
    try:
        cases = [(B.PL_REDUCE_SCATTER, B.PL_ALGO_DIRECT, n // R), (B.PL_REDUCE_SCATTER, B.PL_ALGO_RING, n // R),
                 (B.PL_ALLREDUCE, B.PL_ALGO_ONESHOT, n), (B.PL_ALLREDUCE, B.PL_ALGO_DIRECT_FUSED, n)]
        for coll, algo, n_out in cases:
            s = pl.build(coll, algo, n, 32, hook=hook, out_scale=scale, slice_bytes=16)
            info = B.pl_schedule_info(s)
            f32 = bool(hook & B.PL_HOOK_F32_OUT)
            assert info.hook == hook and info.out_dtype == (B.PL_F32 if f32 else B.PL_BF16)
            for r in range(R):
                assert info.out_bytes[r] == n_out * (4 if f32 else 2)
                assert info.aux_bytes[r] == (n_out * 2 if hook & B.PL_HOOK_RESIDUAL else 0)
            ops = B.pl_schedule_dump(s)
            finals = [o for o in ops if o.dst_bcast & 2]
            assert finals and all(o.kind != B.PL_OP_COPY and o.dst.buf == B.PL_BUF_OUT for o in finals)
            assert all(bool(o.dst_bcast & 2) == (o.dst.buf == B.PL_BUF_OUT) for o in ops)
            assert all(o.dst.dtype == (B.PL_F32 if f32 else B.PL_BF16) for o in finals)
            aux = [gen.normal_bf16(n_out, 5, r) for r in range(R)] if hook & B.PL_HOOK_RESIDUAL else None
            outs = interp_run(ops, info, R, x, seed=3, aux=aux, scale=scale, elem_dtype=B.PL_BF16)
            ref = (oracle.allreduce_processed if coll == B.PL_ALLREDUCE else oracle.reduce_scatter_processed)(x, dtype, scale, aux)
            for r in range(R):
                got = outs[r].view(np.float32).astype(np.float64) if f32 else gen.bf16_bits_to_f64(outs[r].view(np.uint16))
                check_float(got, ref[r], "bf16")
    finally:
        pl.close()


def test_processing_hooks_rejections():
    pl = Planner(4, "bf16")
    try:
        for algo in (B.PL_ALGO_RING, B.PL_ALGO_TREE, B.PL_ALGO_DIRECT):   # all-reduces that end with copies
            with pytest.raises(B.PurlinError) as e:
                pl.build(B.PL_ALLREDUCE, algo, 1024, 256, hook=B.PL_HOOK_RESIDUAL)
            assert e.value.status == B.PL_ERR_UNSUPPORTED
        with pytest.raises(B.PurlinError) as e:
            pl.build(B.PL_ALLGATHER, B.PL_ALGO_DIRECT, 1024, 256, hook=B.PL_HOOK_F32_OUT)
        assert e.value.status == B.PL_ERR_UNSUPPORTED
        with pytest.raises(B.PurlinError) as e:
            pl.build(B.PL_REDUCE_SCATTER, B.PL_ALGO_DIRECT, 1024, 256, hook=8)
        assert e.value.status == B.PL_ERR_INVALID_ARG
        with pytest.raises(B.PurlinError) as e:
            B.pl_schedule_build_layers(pl.comm, B.PL_ALGO_ONESHOT, 1024, 2, B.make_opts(datapath=B.PL_DP_PACKET, hook=B.PL_HOOK_RESIDUAL))
        assert e.value.status == B.PL_ERR_UNSUPPORTED
    finally:
        pl.close()
    for dt, hook in (("i32", B.PL_HOOK_RESIDUAL), ("f32", B.PL_HOOK_F32_OUT)):
        p2 = Planner(4, dt)
        try:
            with pytest.raises(B.PurlinError) as e:
                p2.build(B.PL_REDUCE_SCATTER, B.PL_ALGO_DIRECT, 1024, 256, hook=hook)
            assert e.value.status == B.PL_ERR_UNSUPPORTED
        finally:
            p2.close()


@pytest.mark.parametrize("coll", [B.PL_ALLREDUCE, B.PL_REDUCE_SCATTER, B.PL_ALLGATHER, B.PL_ALLTOALL])
@pytest.mark.parametrize("cap_chunks", [0, 2])
def test_double_buffered_staging_two_overlapped_executes(coll, cap_chunks):
    """Two staging buffers alternated by launch parity (the paper's epoch-parity double buffering):
    the early stage ops of execute B interleave with execute A on the CPU replay; both results must
    be the oracle's, with different inputs per execute."""
    from sched_interp import run_two_overlapped
    R, dtype = 4, "i32"
    chunk = 32
    per = R * 8 * 6 if coll != B.PL_ALLGATHER else 8 * 6
    flags = B.PL_OPT_STAGED | B.PL_OPT_OVERLAP_LAUNCH | B.PL_OPT_STAGE_AHEAD
    pl = Planner(R, dtype)
    try:
        s = pl.build(coll, B.PL_ALGO_DIRECT, per, chunk, flags=flags, staging_bytes=cap_chunks * chunk * (R if coll != B.PL_ALLGATHER else 1),
                     n_ctas=3 * R, slice_bytes=16)
        assert B.pl_schedule_validate(s)[0] == B.PL_OK
        info = B.pl_schedule_info(s)
        ops = B.pl_schedule_dump(s)
        early = [o for o in ops if o.dst_bcast & 4]
        assert early and all(o.kind == B.PL_OP_COPY and o.n_wait == 0 and o.dst.buf == B.PL_BUF_SCRATCH
                             and o.src[0].buf == B.PL_BUF_IN for o in early)
        if cap_chunks:  # cyclic slots: later stage ops wait for their slot and are not early
            assert any(o.kind == B.PL_OP_COPY and o.dst.buf == B.PL_BUF_SCRATCH and not (o.dst_bcast & 4) for o in ops)
        xa = gen.rank_inputs(R, per, dtype)
        xb = [(a.astype(np.int64) * 3 + 11).astype(np.int32) for a in xa]
        got_a, got_b, early_steps = run_two_overlapped(ops, info, R, xa, xb, seed=4)
        assert early_steps > 0
        fn = {B.PL_ALLREDUCE: lambda x: oracle.allreduce(x, dtype), B.PL_REDUCE_SCATTER: lambda x: oracle.reduce_scatter(x, dtype),
              B.PL_ALLGATHER: oracle.allgather, B.PL_ALLTOALL: oracle.alltoall}[coll]
        for got, x in ((got_a, xa), (got_b, xb)):
            ref = fn(x)
            for r in range(R):
                assert np.array_equal(got[r].view(np.int32), np.asarray(ref[r]).view(np.int32))
    finally:
        pl.close()


def test_stage_ahead_needs_staging_and_overlapped_launches():
    pl = Planner(4, "bf16")
    try:
        for flags in (B.PL_OPT_STAGE_AHEAD, B.PL_OPT_STAGE_AHEAD | B.PL_OPT_STAGED, B.PL_OPT_STAGE_AHEAD | B.PL_OPT_OVERLAP_LAUNCH,
                      B.PL_OPT_STAGE_AHEAD | B.PL_OPT_STAGED | B.PL_OPT_OVERLAP_LAUNCH | B.PL_OPT_TRACE):
            with pytest.raises(B.PurlinError) as e:
                pl.build(B.PL_ALLREDUCE, B.PL_ALGO_DIRECT, 1024, 256, flags=flags)
            assert e.value.status == B.PL_ERR_INVALID_ARG
        s = pl.build(B.PL_ALLREDUCE, B.PL_ALGO_DIRECT, 1024, 256, flags=B.PL_OPT_STAGED | B.PL_OPT_OVERLAP_LAUNCH | B.PL_OPT_STAGE_AHEAD)
        one = pl.build(B.PL_ALLREDUCE, B.PL_ALGO_DIRECT, 1024, 256, flags=B.PL_OPT_STAGED | B.PL_OPT_OVERLAP_LAUNCH)
        assert B.pl_schedule_info(s).scratch_bytes == 2 * B.pl_schedule_info(one).scratch_bytes   # two staging buffers
    finally:
        pl.close()


def test_hbm_bytes_count_every_input_byte_once():
    """pl_sched_info_t.hbm_bytes: bytes_read with the caller's inputs counted once, plus bytes_written."""
    R, M = 8, 1 << 20            # bf16, 1 MiB per rank
    pl = Planner(R, "bf16")
    try:
        n = M // 2
        want = {
            (B.PL_REDUCE_SCATTER, B.PL_ALGO_DIRECT, n): (R + 1) * M,                 # read everything once, write M / R per rank
            (B.PL_ALLGATHER, B.PL_ALGO_DIRECT, n // R): (R + 1) * M,                 # contributions once, R * M written
            (B.PL_ALLGATHER, B.PL_ALGO_RING, n // R): (R + 1) * M + (R - 2) * M,      # + what the hops re-read from outputs
            (B.PL_ALLREDUCE, B.PL_ALGO_ONESHOT, n): 2 * R * M,                       # inputs once (not R times), R * M written
            (B.PL_ALLREDUCE, B.PL_ALGO_DIRECT_FUSED, n): 2 * R * M,
            (B.PL_ALLREDUCE, B.PL_ALGO_DIRECT, n): R * M + M + (R - 1) * M + (R - 1) * M,  # + reduced partitions re-read by R - 1 ranks
            (B.PL_ALLTOALL, B.PL_ALGO_DIRECT, n): 2 * R * M,
        }
        for (coll, algo, count), bytes_ in want.items():
            info = B.pl_schedule_info(pl.build(coll, algo, count, 65536, datapath=B.PL_DP_TMA))
            assert info.hbm_bytes == bytes_, (coll, algo, info.hbm_bytes, bytes_)
            assert info.hbm_bytes <= info.bytes_read + info.bytes_written
        # ring reduce-scatter: every input partition once (the chain start reads two inputs of the same
        # partition from two ranks), the travelling fp32 partials written and read once per hop
        info = B.pl_schedule_info(pl.build(B.PL_REDUCE_SCATTER, B.PL_ALGO_RING, n, 65536, datapath=B.PL_DP_TMA))
        P = M // R
        assert info.hbm_bytes == R * M + 2 * R * (R - 2) * 2 * P + R * P
    finally:
        pl.close()


def test_config1_op_counts_and_bytes():
    # all-reduce, R=4, 262144 fp32 per rank, ring, 64 KiB chunks, unsliced:
    # 3 reduce-scatter hops + 3 all-gather hops, 4 ranks, 4 chunks per partition
    pl = Planner(4, "f32")
    try:
        s = pl.build(B.PL_ALLREDUCE, B.PL_ALGO_RING, 262144, 65536, slice_bytes=131072)
        info = B.pl_schedule_info(s)
        ops = B.pl_schedule_dump(s)
        assert sum(o.kind == B.PL_OP_COPY_REDUCE for o in ops) == 48
        assert sum(o.kind == B.PL_OP_COPY for o in ops) == 48
        M = 1 << 20
        # fp32 partials travel as (sum, correction) pairs: per partition element the three
        # reduce-scatter hops move 16 + 20 + 16 bytes, the all-gather hops 2 * 4 * 3
        assert info.bytes_read + info.bytes_written == 13 * M + 6 * M
        assert info.message_bytes == M
    finally:
        pl.close()
    pl = Planner(4, "i32")
    try:
        s = pl.build(B.PL_ALLREDUCE, B.PL_ALGO_RING, 262144, 65536, slice_bytes=65536)
        info = B.pl_schedule_info(s)
        assert info.bytes_read + info.bytes_written == 5 * 3 * (1 << 20)  # 5(R-1)M with same-width partials
    finally:
        pl.close()


def test_schedule_bytes_match_closed_forms_bf16_R8():
    R, M = 8, 1 << 20
    n = M // 2
    pl = Planner(R, "bf16")
    try:
        def total(coll, algo, count=n, **kw):
            i = B.pl_schedule_info(pl.build(coll, algo, count, 1 << 16, **kw))
            return i.bytes_read + i.bytes_written
        assert total(B.PL_REDUCE_SCATTER, B.PL_ALGO_DIRECT) == (R + 1) * M
        assert total(B.PL_REDUCE_SCATTER, B.PL_ALGO_RING) == 33 * M  # fp32 partials: (16+10(R-3))/2 per byte
        # per-rank-message M = gathered size; the direct all-gather is a push on both datapaths: each
        # contribution is read once and written R times; the ring copies it hop by hop
        assert total(B.PL_ALLGATHER, B.PL_ALGO_DIRECT, n // R, datapath=B.PL_DP_TMA) == (R + 1) * M
        assert total(B.PL_ALLGATHER, B.PL_ALGO_DIRECT, n // R, datapath=B.PL_DP_LDST) == (R + 1) * M
        assert total(B.PL_ALLGATHER, B.PL_ALGO_RING, n // R) == 2 * R * M
        assert total(B.PL_ALLREDUCE, B.PL_ALGO_ONESHOT) == R * (R + 1) * M
        assert total(B.PL_ALLREDUCE, B.PL_ALGO_DIRECT) == (3 * R - 1) * M
        assert total(B.PL_ALLREDUCE, B.PL_ALGO_DIRECT_FUSED) == 2 * R * M
        assert total(B.PL_ALLREDUCE, B.PL_ALGO_RING) == 47 * M
        assert total(B.PL_ALLREDUCE, B.PL_ALGO_TREE) == 47 * M
    finally:
        pl.close()


def test_error_rules():
    with pytest.raises(B.PurlinError) as e:
        B.pl_comm_create_planner(1, B.PL_BF16)
    assert e.value.status == B.PL_ERR_INVALID_ARG
    with pytest.raises(B.PurlinError):
        B.pl_comm_create_planner(17, B.PL_BF16)
    pl = Planner(8, "bf16")
    try:
        def status(fn):
            with pytest.raises(B.PurlinError) as ei:
                fn()
            return ei.value.status
        # bytes not divisible by R*16
        assert status(lambda: pl.build(B.PL_REDUCE_SCATTER, B.PL_ALGO_DIRECT, 8 * 8 + 8, 64)) == B.PL_ERR_INVALID_ARG
        assert "divisible by 16*R" in B.pl_comm_last_error(pl.comm)
        # chunk not a multiple of 16 / zero
        assert status(lambda: pl.build(B.PL_ALLREDUCE, B.PL_ALGO_DIRECT, 1024, 24)) == B.PL_ERR_INVALID_ARG
        assert status(lambda: pl.build(B.PL_ALLREDUCE, B.PL_ALGO_DIRECT, 1024, 0)) == B.PL_ERR_INVALID_ARG
        # tree on a non-allreduce, fused all-gather
        assert status(lambda: pl.build(B.PL_REDUCE_SCATTER, B.PL_ALGO_TREE, 1024, 64)) == B.PL_ERR_UNSUPPORTED
        assert status(lambda: pl.build(B.PL_ALLGATHER, B.PL_ALGO_DIRECT_FUSED, 1024, 64)) == B.PL_ERR_UNSUPPORTED
        assert status(lambda: pl.build(B.PL_ALLTOALL, B.PL_ALGO_RING, 1024, 64)) == B.PL_ERR_UNSUPPORTED
        # more CTAs than can be co-resident
        assert status(lambda: pl.build(B.PL_ALLREDUCE, B.PL_ALGO_DIRECT, 1 << 20, 1 << 16, n_ctas=100000)) == B.PL_ERR_OVERSUBSCRIBED
        # all-to-all-v segment not 16-byte aligned
        C = [[4] * 8 for _ in range(8)]
        assert status(lambda: B.pl_schedule_build_v(pl.comm, B.PL_ALLTOALLV, B.PL_ALGO_DIRECT, C, 64)) == B.PL_ERR_ALIGNMENT
        # planner communicators cannot execute
        s = pl.build(B.PL_ALLREDUCE, B.PL_ALGO_DIRECT, 1024, 64)
        bufs = B.make_bufs([16] * 8, [16] * 8, [1 << 20] * 8, [1 << 20] * 8)
        assert status(lambda: B.pl_execute(s, bufs)) == B.PL_ERR_UNSUPPORTED
        # layered schedules: ring is not offered
        assert status(lambda: B.pl_schedule_build_layers(pl.comm, B.PL_ALGO_RING, 1024, 4)) == B.PL_ERR_UNSUPPORTED
        # a communicator with live schedules cannot be destroyed
        assert status(lambda: B.pl_comm_destroy(pl.comm)) == B.PL_ERR_INVALID_ARG
    finally:
        pl.close()
    plu = Planner(4, "u8")
    try:
        with pytest.raises(B.PurlinError) as ei:
            plu.build(B.PL_ALLREDUCE, B.PL_ALGO_DIRECT, 1024, 64)
        assert ei.value.status == B.PL_ERR_UNSUPPORTED
    finally:
        plu.close()


def test_validator_catches_a_broken_edge():
    # raising one wait's needed count makes the replay deadlock: the interpreter notices
    pl = Planner(4, "i32")
    try:
        n = 4 * 4 * 4
        s = pl.build(B.PL_ALLREDUCE, B.PL_ALGO_RING, n, 16)
        ops = B.pl_schedule_dump(s)
        victim = next(o for o in ops if o.n_wait > 0)
        victim.wait_need[0] += 1
        with pytest.raises(AssertionError):
            interp_run(ops, B.pl_schedule_info(s), 4, gen.rank_coded_i32(4, n))
    finally:
        pl.close()


def test_queues_are_rank_owned_and_balanced():
    pl = Planner(8, "bf16")
    try:
        s = pl.build(B.PL_REDUCE_SCATTER, B.PL_ALGO_DIRECT, 8 << 20, 1 << 20, n_ctas=144)  # automatic slicing
        ops = B.pl_schedule_dump(s)
        load = {}
        for o in ops:
            assert o.queue % 8 == o.exec_rank
            load[o.queue] = load.get(o.queue, 0) + o.count
        assert len(load) == 144
        assert max(load.values()) <= 1.25 * min(load.values())
    finally:
        pl.close()


# ---- staged schedules: ordinary application buffers, cyclic staging, role-specialised queues ----
@pytest.mark.parametrize("R", [2, 3, 8])
@pytest.mark.parametrize("cap_chunks", [1, 2, 100])
def test_staged_collectives_replay_to_oracle(R, cap_chunks):
    chunk = 48
    for dtype in ("i32", "bf16"):
        es = B.DTYPE_SIZE[DT[dtype]]
        n = R * (16 // es) * 13                     # 13 vectors per partition: 5 chunks of 48 B, last one short
        x = gen.rank_inputs(R, n, dtype, seed=R + 1)
        pl = Planner(R, dtype)
        try:
            kw = dict(flags=B.PL_OPT_STAGED, staging_bytes=cap_chunks * R * chunk, slice_bytes=32, n_ctas=6 * R)
            s = pl.build(B.PL_ALLREDUCE, B.PL_ALGO_DIRECT, n, chunk, **kw)
            st, msg = B.pl_schedule_validate(s)
            assert st == B.PL_OK, msg
            info = B.pl_schedule_info(s)
            ops = B.pl_schedule_dump(s)
            # nothing but the staging copies reads an input, nothing but the rank itself reads it
            for o in ops:
                for k in range(o.n_src):
                    if o.src[k].buf == B.PL_BUF_IN:
                        assert o.kind == B.PL_OP_COPY and o.src[k].rank == o.exec_rank and o.dst.buf == B.PL_BUF_SCRATCH
                if o.dst.buf == B.PL_BUF_OUT:
                    assert o.dst.rank == o.exec_rank
            if cap_chunks < 5:
                # cyclic staging: scratch is smaller than the message and some stage op waits
                assert info.scratch_bytes < R * (n * es + n * es // R)
                assert any(o.n_wait > 0 and o.dst.buf == B.PL_BUF_SCRATCH and o.kind == B.PL_OP_COPY for o in ops)
            for seed in (0, 1, 2):
                compare_reduce(interp_run(ops, info, R, x, seed=seed), oracle.allreduce(x, dtype), dtype)
            s = pl.build(B.PL_REDUCE_SCATTER, B.PL_ALGO_DIRECT, n, chunk, **kw)
            assert B.pl_schedule_validate(s)[0] == B.PL_OK
            compare_reduce(interp_run(B.pl_schedule_dump(s), B.pl_schedule_info(s), R, x, seed=3),
                           oracle.reduce_scatter(x, dtype), dtype)
            kw_ag = dict(kw, staging_bytes=cap_chunks * chunk)
            s = pl.build(B.PL_ALLGATHER, B.PL_ALGO_DIRECT, n, chunk, **kw_ag)
            assert B.pl_schedule_validate(s)[0] == B.PL_OK
            outs = interp_run(B.pl_schedule_dump(s), B.pl_schedule_info(s), R, x, seed=4)
            ref = oracle.allgather(x)
            for r in range(R):
                assert np.array_equal(outs[r], ref[r].view(np.uint8))
            s = pl.build(B.PL_ALLTOALL, B.PL_ALGO_DIRECT, n, chunk, **kw)
            assert B.pl_schedule_validate(s)[0] == B.PL_OK
            outs = interp_run(B.pl_schedule_dump(s), B.pl_schedule_info(s), R, x, seed=5)
            ref = oracle.alltoall(x)
            for r in range(R):
                assert np.array_equal(outs[r], ref[r].view(np.uint8))
        finally:
            pl.close()


def test_staged_roles_get_their_own_queues():
    R = 8
    pl = Planner(R, "bf16")
    try:
        s = pl.build(B.PL_ALLREDUCE, B.PL_ALGO_DIRECT, 8 << 20, 1 << 20, flags=B.PL_OPT_STAGED, n_ctas=144)
        ops = B.pl_schedule_dump(s)
        kinds = {}
        for o in ops:
            role = "stage" if o.dst.buf == B.PL_BUF_SCRATCH and o.kind == B.PL_OP_COPY else \
                   "reduce" if o.kind == B.PL_OP_REDUCE else "gather"
            kinds.setdefault(o.queue, set()).add(role)
        assert all(len(v) == 1 for v in kinds.values())       # a queue serves one role only
        per_role = {}
        for q, v in kinds.items():
            if q % R == 0:
                per_role[next(iter(v))] = per_role.get(next(iter(v)), 0) + 1
        assert sum(per_role.values()) == 18 and per_role["stage"] >= 6 and per_role["gather"] >= 6 and per_role["reduce"] >= 3
    finally:
        pl.close()


def test_staged_rejections():
    pl = Planner(4, "bf16")
    try:
        for coll, algo in ((B.PL_ALLREDUCE, B.PL_ALGO_RING), (B.PL_ALLREDUCE, B.PL_ALGO_ONESHOT), (B.PL_REDUCE_SCATTER, B.PL_ALGO_RING)):
            with pytest.raises(B.PurlinError) as e:
                pl.build(coll, algo, 4096, 256, flags=B.PL_OPT_STAGED)
            assert e.value.status == B.PL_ERR_UNSUPPORTED
    finally:
        pl.close()


def test_validator_notices_a_dropped_wait_edge():
    pl = Planner(4, "i32")
    try:
        n = 4 * 4 * 6
        # a ring: dropping the wait of a hop leaves a read of the travelling partial unordered
        s = pl.build(B.PL_ALLREDUCE, B.PL_ALGO_RING, n, 32)
        assert B.pl_schedule_validate(s)[0] == B.PL_OK
        victim = next(o.topo for o in B.pl_schedule_dump(s) if o.n_wait > 0)
        B.pl_schedule_debug_drop_wait(s, victim)
        st, msg = B.pl_schedule_validate(s)
        assert st == B.PL_ERR_INVALID_SCHEDULE and "without being ordered" in msg
        # cyclic staging: dropping the "slot is free again" wait of a stage op is a write-after-read hazard
        s = pl.build(B.PL_ALLREDUCE, B.PL_ALGO_DIRECT, n, 32, flags=B.PL_OPT_STAGED, staging_bytes=4 * 32)
        assert B.pl_schedule_validate(s)[0] == B.PL_OK
        # one slot of 32 bytes per partition: the slot of partition k starts at byte 32*k; take a
        # stage op whose consumer is another rank (on the same rank queue order would still protect it)
        victim = next(o.topo for o in B.pl_schedule_dump(s)
                      if o.n_wait > 0 and o.kind == B.PL_OP_COPY and o.dst.buf == B.PL_BUF_SCRATCH
                      and o.dst.offset // 32 != o.exec_rank)
        B.pl_schedule_debug_drop_wait(s, victim)
        st, msg = B.pl_schedule_validate(s)
        assert st == B.PL_ERR_INVALID_SCHEDULE and "overwrites scratch" in msg
    finally:
        pl.close()


def test_validator_counts_queue_order_only_where_the_executor_gives_it():
    """The register executor finishes an op before the next one of its queue starts; the bulk-copy
    executor issues later ops' loads ahead of earlier ops' stores.  A read-after-write on one queue
    with no flag edge is therefore fine for the first and must be rejected for the second."""
    pl = Planner(4, "i32")
    try:
        n = 4 * 4 * 8
        for datapath, want in ((B.PL_DP_LDST, B.PL_OK), (B.PL_DP_TMA, B.PL_ERR_INVALID_SCHEDULE)):
            # tree with one queue per rank: a rank's level-1 addition reads its own level-0 partial
            s = pl.build(B.PL_ALLREDUCE, B.PL_ALGO_TREE, n, n * 4, n_ctas=4, datapath=datapath)
            assert B.pl_schedule_validate(s)[0] == B.PL_OK
            ops = B.pl_schedule_dump(s)
            signaller = {o.signal_flag: o for o in ops if o.signal_flag >= 0}
            victim = next(o.topo for o in ops if o.kind == B.PL_OP_COPY_REDUCE and o.n_wait == 2
                          and signaller[o.wait_flag[0]].queue == o.queue)
            B.pl_schedule_debug_drop_wait(s, victim)
            st, msg = B.pl_schedule_validate(s)
            assert st == want, msg
            if want != B.PL_OK:
                assert "without being ordered" in msg
    finally:
        pl.close()


@pytest.mark.parametrize("R", [2, 3, 8])
def test_every_lowering_validates_under_the_bulk_copy_rules(R):
    """All algorithms carry explicit flag edges for every dependency the bulk-copy executor does
    not give by queue order (build runs the validator; a failure would raise)."""
    pl = Planner(R, "bf16")
    try:
        n = R * 8 * 24
        for chunk in (16, 64, n * 2):
            for nct in (R, 3 * R):
                kw = dict(datapath=B.PL_DP_TMA, n_ctas=nct, slice_bytes=32)
                for algo in ALLREDUCE_ALGOS:
                    pl.build(B.PL_ALLREDUCE, algo, n, chunk, **kw)
                for coll in (B.PL_REDUCE_SCATTER, B.PL_ALLGATHER):
                    for algo in (B.PL_ALGO_DIRECT, B.PL_ALGO_RING):
                        pl.build(coll, algo, n, chunk, **kw)
                pl.build(B.PL_ALLTOALL, B.PL_ALGO_DIRECT, n, chunk, **kw)
                for coll in (B.PL_ALLREDUCE, B.PL_REDUCE_SCATTER, B.PL_ALLGATHER, B.PL_ALLTOALL):
                    pl.build(coll, B.PL_ALGO_DIRECT, n, chunk, flags=B.PL_OPT_STAGED, staging_bytes=2 * chunk * R, **kw)
    finally:
        pl.close()


# ---- V variants of all-gather / reduce-scatter ---------------------------------------------
@pytest.mark.parametrize("R", [2, 5, 8])
def test_allgatherv_reduce_scatterv_replay(R):
    rng = np.random.default_rng(R)
    sizes = (rng.integers(0, 6, size=R) * 8).tolist()      # elements; zero-size partitions included
    sizes[0] = 40
    total = sum(sizes)
    for dtype in ("i32", "bf16"):
        es = B.DTYPE_SIZE[DT[dtype]]
        pl = Planner(R, dtype)
        try:
            x = gen.rank_inputs(R, total, dtype, seed=3)
            s = B.pl_schedule_build_v(pl.comm, B.PL_REDUCE_SCATTERV, B.PL_ALGO_DIRECT, sizes, 48, B.make_opts(slice_bytes=32))
            pl.scheds.append(s)
            info = B.pl_schedule_info(s)
            assert B.pl_schedule_validate(s)[0] == B.PL_OK
            assert info.message_bytes == total * es
            assert [int(info.out_bytes[r]) for r in range(R)] == [n * es for n in sizes]
            outs = interp_run(B.pl_schedule_dump(s), info, R, x, seed=1)
            ref = oracle.reduce_scatterv(x, sizes, dtype)
            for r in range(R):
                o = outs[r]
                if dtype == "i32":
                    assert np.array_equal(o.view(np.int32), ref[r])
                else:
                    check_float(gen.bf16_bits_to_f64(o.view(np.uint16)), ref[r], dtype)
            contrib = [x[p][: sizes[p]].copy() for p in range(R)]
            s = B.pl_schedule_build_v(pl.comm, B.PL_ALLGATHERV, B.PL_ALGO_DIRECT, sizes, 48, B.make_opts(slice_bytes=32))
            pl.scheds.append(s)
            info = B.pl_schedule_info(s)
            assert [int(info.in_bytes[r]) for r in range(R)] == [n * es for n in sizes]
            outs = interp_run(B.pl_schedule_dump(s), info, R, [c if c.size else np.zeros(0, c.dtype) for c in contrib], seed=2)
            ref = oracle.allgatherv(contrib)
            for r in range(R):
                assert np.array_equal(outs[r], ref[r].view(np.uint8))
        finally:
            pl.close()
    pl = Planner(4, "bf16")
    try:
        with pytest.raises(B.PurlinError) as e:
            B.pl_schedule_build_v(pl.comm, B.PL_ALLGATHERV, B.PL_ALGO_DIRECT, [8, 4, 8, 8], 64)
        assert e.value.status == B.PL_ERR_ALIGNMENT
        with pytest.raises(B.PurlinError) as e:
            B.pl_schedule_build_v(pl.comm, B.PL_REDUCE_SCATTERV, B.PL_ALGO_RING, [8, 8, 8, 8], 64)
        assert e.value.status == B.PL_ERR_UNSUPPORTED
    finally:
        pl.close()


# ---- rooted collectives -----------------------------------------------------------------------
@pytest.mark.parametrize("R,root", [(2, 1), (5, 0), (8, 3)])
def test_rooted_collectives_replay(R, root):
    for dtype in ("i32", "bf16"):
        es = B.DTYPE_SIZE[DT[dtype]]
        m = (16 // es) * 7
        n = R * m
        x = gen.rank_inputs(R, n, dtype, seed=17)
        empty = np.zeros(0, x[0].dtype)
        pl = Planner(R, dtype)
        try:
            def build(coll, count):
                s = B.pl_schedule_build_rooted(pl.comm, coll, root, count, 48, B.make_opts(slice_bytes=32, n_ctas=2 * R))
                pl.scheds.append(s)
                st, msg = B.pl_schedule_validate(s)
                assert st == B.PL_OK, msg
                return s, B.pl_schedule_info(s)
            s, info = build(B.PL_BROADCAST, n)
            assert [int(info.in_bytes[r]) for r in range(R)] == [n * es if r == root else 0 for r in range(R)]
            outs = interp_run(B.pl_schedule_dump(s), info, R, [x[r] if r == root else empty for r in range(R)], seed=1)
            for r in range(R):
                assert np.array_equal(outs[r], oracle.broadcast(x, root)[r].view(np.uint8))
            s, info = build(B.PL_REDUCE, n)
            assert [int(info.out_bytes[r]) for r in range(R)] == [n * es if r == root else 0 for r in range(R)]
            outs = interp_run(B.pl_schedule_dump(s), info, R, x, seed=2)
            ref = oracle.reduce(x, root, dtype)[root]
            if dtype == "i32":
                assert np.array_equal(outs[root].view(np.int32), ref)
            else:
                check_float(gen.bf16_bits_to_f64(outs[root].view(np.uint16)), ref, dtype)
            s, info = build(B.PL_SCATTER, m)
            outs = interp_run(B.pl_schedule_dump(s), info, R, [x[r] if r == root else empty for r in range(R)], seed=3)
            for r in range(R):
                assert np.array_equal(outs[r], oracle.scatter(x, root)[r].view(np.uint8))
            contrib = [a[:m].copy() for a in x]
            s, info = build(B.PL_GATHER, m)
            outs = interp_run(B.pl_schedule_dump(s), info, R, contrib, seed=4)
            assert np.array_equal(outs[root], oracle.gather(contrib, root)[root].view(np.uint8))
            assert all(outs[r].size == 0 for r in range(R) if r != root)
            with pytest.raises(B.PurlinError):
                B.pl_schedule_build_rooted(pl.comm, B.PL_BROADCAST, R, n, 48, None)
            with pytest.raises(B.PurlinError):
                B.pl_schedule_build_rooted(pl.comm, B.PL_ALLREDUCE, 0, n, 48, None)
        finally:
            pl.close()


def test_tree_root_rotates_with_the_chunk_and_balances_the_ranks():
    """Binomial tree: 2(R-1) ops per chunk over log2(R) + log2(R) stages; the op that writes the
    reduced chunk (the root's) moves to rank c mod R with the chunk index, so every rank carries
    the same bytes when the chunk count is a multiple of R; one chunk is the rank-0 tree."""
    R, es = 8, 4
    pl = Planner(R, "i32")
    try:
        n = 16 * 256  # 16 chunks of 1 KiB
        s = pl.build(B.PL_ALLREDUCE, B.PL_ALGO_TREE, n, 1024, n_ctas=R, slice_bytes=1 << 20)
        ops = B.pl_schedule_dump(s)
        assert len(ops) == 16 * 2 * (R - 1)
        roots = {}
        per_rank = [0] * R
        for o in ops:
            per_rank[o.exec_rank] += o.count * (es if o.kind != B.PL_OP_COPY else 1)
            if o.kind == B.PL_OP_COPY_REDUCE and o.dst.buf == B.PL_BUF_OUT:
                roots[int(o.dst.offset) // 1024] = o.exec_rank
        assert roots == {c: c % R for c in range(16)}
        assert len(set(per_rank)) == 1
        # a single chunk: reduce ends on rank 0, which never receives a broadcast copy
        s1 = pl.build(B.PL_ALLREDUCE, B.PL_ALGO_TREE, 256, 1024, n_ctas=R, slice_bytes=1 << 20)
        ops1 = B.pl_schedule_dump(s1)
        assert len(ops1) == 2 * (R - 1)
        assert [o.exec_rank for o in ops1 if o.kind == B.PL_OP_COPY_REDUCE and o.dst.buf == B.PL_BUF_OUT] == [0]
        assert sorted(o.exec_rank for o in ops1 if o.kind == B.PL_OP_COPY) == list(range(1, R))
    finally:
        pl.close()


def test_latency_regime_grid_follows_the_schedule_width():
    """Small messages with the grid left to the library: a rank gets one queue per op it can run
    at the same depth of the dependency graph (two-shot all-reduce: R - 1 gather copies)."""
    R = 8
    pl = Planner(R, "bf16")
    try:
        s = pl.build(B.PL_ALLREDUCE, B.PL_ALGO_DIRECT, 2048, 512)  # 4 KiB per rank
        info = B.pl_schedule_info(s)
        ops = B.pl_schedule_dump(s)
        assert info.n_queues == R * (R - 1)
        # no queue holds two ops of the same phase
        seen = set()
        for o in ops:
            key = (o.queue, o.kind)
            assert key not in seen
            seen.add(key)
    finally:
        pl.close()


def test_algo_auto_picks_by_collective_and_size():
    """PL_ALGO_AUTO: one-shot for all-reduces up to 32 KiB per rank, direct-fused above, direct for
    everything else; the schedules are the same as the explicitly named ones."""
    R = 8
    pl = Planner(R, "bf16")
    try:
        def same(coll, count, named):
            a = B.pl_schedule_dump(pl.build(coll, B.PL_ALGO_AUTO, count, 1 << 20))
            b = B.pl_schedule_dump(pl.build(coll, named, count, 1 << 20))
            key = lambda o: (o.kind, o.exec_rank, o.queue, int(o.count), int(o.dst.offset), o.n_src, o.dst_bcast)
            assert [key(o) for o in a] == [key(o) for o in b]
        same(B.PL_ALLREDUCE, 8192, B.PL_ALGO_ONESHOT)           # 16 KiB
        same(B.PL_ALLREDUCE, 16384, B.PL_ALGO_ONESHOT)          # 32 KiB
        same(B.PL_ALLREDUCE, 32768, B.PL_ALGO_DIRECT_FUSED)     # 64 KiB
        same(B.PL_ALLREDUCE, 1 << 24, B.PL_ALGO_DIRECT_FUSED)
        same(B.PL_REDUCE_SCATTER, 1 << 20, B.PL_ALGO_DIRECT)
        same(B.PL_ALLGATHER, 1 << 17, B.PL_ALGO_DIRECT)
        same(B.PL_ALLTOALL, 1 << 20, B.PL_ALGO_DIRECT)
        s = B.pl_schedule_build_layers(pl.comm, B.PL_ALGO_AUTO, 8192, 4, None)
        pl.scheds.append(s)
        assert all(o.dst_bcast for o in B.pl_schedule_dump(s))  # direct-fused layers
    finally:
        pl.close()


def test_pushed_all_gather_default_grid_and_option_flags_on_the_planner():
    """Policy, no GPU: the pushed all-gather of the bulk-copy datapath asks for fewer CTAs than a
    reduce-scatter of the same size (a 1 read : R writes stream wants fewer writers), a multiple
    of R either way; the L2 options change nothing in what is lowered; tuning needs a GPU."""
    R = 8
    pl = Planner(R, "bf16")
    try:
        n = R * (4 << 20)
        ag = pl.build(B.PL_ALLGATHER, B.PL_ALGO_DIRECT, n // R, 1 << 20, datapath=B.PL_DP_TMA)
        rs = pl.build(B.PL_REDUCE_SCATTER, B.PL_ALGO_DIRECT, n, 1 << 20, datapath=B.PL_DP_TMA)
        ia, ir = B.pl_schedule_info(ag), B.pl_schedule_info(rs)
        assert ia.grid % R == 0 and ir.grid % R == 0
        assert ia.grid < ir.grid and 0.80 * ir.grid <= ia.grid <= 0.90 * ir.grid
        plain = B.pl_schedule_dump(rs)
        for flags in (B.PL_OPT_INPUTS_LAST_USE, B.PL_OPT_NO_L2_HINTS, B.PL_OPT_INPUTS_LAST_USE | B.PL_OPT_NO_L2_HINTS):
            s = pl.build(B.PL_REDUCE_SCATTER, B.PL_ALGO_DIRECT, n, 1 << 20, datapath=B.PL_DP_TMA, flags=flags)
            i2 = B.pl_schedule_info(s)
            assert (i2.grid, i2.n_ops, i2.bytes_read, i2.bytes_written, i2.hbm_bytes) == (ir.grid, ir.n_ops, ir.bytes_read, ir.bytes_written, ir.hbm_bytes)
            ops = B.pl_schedule_dump(s)
            assert [(o.kind, o.queue, o.count) for o in ops] == [(o.kind, o.queue, o.count) for o in plain]
        with pytest.raises(B.PurlinError) as e:
            B.pl_comm_tune(pl.comm, 0)
        assert e.value.status == B.PL_ERR_UNSUPPORTED
    finally:
        pl.close()
