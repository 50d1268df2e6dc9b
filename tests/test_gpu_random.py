"""Randomised parity on the GPU: seeded draws of communicator size, element type, collective,
algorithm, message, chunk and slice sizes, grid and datapath; every case is executed twice on
poisoned outputs and compared with the oracle element by element (bit-exact for integers and
copies, spec tolerance for floats).  Sizes stay small (the oracle finishes in
milliseconds) but are ragged against chunks, slices and the 48 KiB ring slots."""
import numpy as np
import pytest

from oracle import oracle
from paper_2609_36954_b200 import binding as B
from paper_2609_36954_b200 import inputs as gen

from gpu_harness import DT, Session, check_float

pytestmark = pytest.mark.gpu

ALGOS = {
    B.PL_ALLREDUCE: [B.PL_ALGO_RING, B.PL_ALGO_TREE, B.PL_ALGO_DIRECT, B.PL_ALGO_ONESHOT, B.PL_ALGO_DIRECT_FUSED],
    B.PL_REDUCE_SCATTER: [B.PL_ALGO_RING, B.PL_ALGO_DIRECT],
    B.PL_ALLGATHER: [B.PL_ALGO_RING, B.PL_ALGO_DIRECT],
    B.PL_ALLTOALL: [B.PL_ALGO_DIRECT],
}


def draw(rng):
    R = int(rng.choice([2, 3, 4, 5, 7, 8, 12, 16]))
    dtype = str(rng.choice(["i32", "bf16", "f32"]))
    coll = int(rng.choice(list(ALGOS)))
    algo = int(rng.choice(ALGOS[coll]))
    staged = bool(rng.integers(0, 4) == 0) and algo == B.PL_ALGO_DIRECT
    vecs = int(rng.choice([1, 3, 17, 64, 257, 1031, 4099]))        # 16-byte vectors per partition
    chunk_vecs = int(rng.choice([1, 5, 64, 512, 3000, 1 << 20]))
    slice_vecs = int(rng.choice([0, 0, 1, 7, 128, 1024]))
    queues = int(rng.choice([0, 1, 2, 5, 9]))
    dp = int(rng.choice([B.PL_DP_AUTO, B.PL_DP_LDST, B.PL_DP_TMA]))
    return dict(R=R, dtype=dtype, coll=coll, algo=algo, staged=staged, vecs=vecs, chunk_vecs=chunk_vecs,
                slice_vecs=slice_vecs, queues=queues, dp=dp)


@pytest.mark.parametrize("seed", range(96))
def test_random_case_matches_the_oracle(seed):
    rng = np.random.default_rng(1000 + seed)
    c = draw(rng)
    R, dtype, coll = c["R"], c["dtype"], c["coll"]
    es = B.DTYPE_SIZE[DT[dtype]]
    n = R * c["vecs"] * (16 // es)
    count = n // R if coll == B.PL_ALLGATHER else n
    s = Session(R, dtype)
    try:
        kw = dict(slice_bytes=16 * c["slice_vecs"], datapath=c["dp"], n_ctas=c["queues"] * R)
        if c["staged"]:
            kw.update(flags=B.PL_OPT_STAGED, staging_bytes=(R if coll != B.PL_ALLGATHER else 1) * 16 * min(c["chunk_vecs"], c["vecs"]) * 2)
        sched = s.build(coll, c["algo"], count, 16 * c["chunk_vecs"], **kw)
        x = gen.rank_inputs(R, n, dtype, seed=seed)
        if coll == B.PL_ALLGATHER:
            x = [a[:count].copy() for a in x]
        outs, _ = s.execute(sched, x, repeats=2)
        if coll == B.PL_ALLREDUCE:
            ref = oracle.allreduce(x, dtype)
        elif coll == B.PL_REDUCE_SCATTER:
            ref = oracle.reduce_scatter(x, dtype)
        elif coll == B.PL_ALLGATHER:
            ref = oracle.allgather(x)
        else:
            ref = oracle.alltoall(x)
        for r in range(R):
            if coll in (B.PL_ALLGATHER, B.PL_ALLTOALL) or dtype == "i32":
                assert np.array_equal(outs[r], np.ascontiguousarray(ref[r]).view(np.uint8).reshape(-1)), (c, r)
            elif dtype == "bf16":
                check_float(gen.bf16_bits_to_f64(outs[r].view(np.uint16)), ref[r], dtype)
            else:
                check_float(outs[r].view(np.float32).astype(np.float64), ref[r], dtype)
    finally:
        s.close()


@pytest.mark.parametrize("seed", range(48))
def test_random_v_and_rooted_case_matches_the_oracle(seed):
    """Seeded draws for the variable-size collectives (ragged per-rank sizes with empty ranks)
    and the rooted ones (any root), over rank count, element type, chunk size and datapath."""
    rng = np.random.default_rng(7000 + seed)
    R = int(rng.choice([2, 3, 5, 8, 11, 16]))
    dtype = str(rng.choice(["i32", "bf16", "f32"]))
    es = B.DTYPE_SIZE[DT[dtype]]
    dp = int(rng.choice([B.PL_DP_AUTO, B.PL_DP_LDST, B.PL_DP_TMA]))
    chunk = 16 * int(rng.choice([1, 7, 256, 4096, 1 << 16]))
    kind = str(rng.choice(["agv", "rsv", "a2av", "broadcast", "reduce", "scatter", "gather"]))
    vec = 16 // es
    s = Session(R, dtype)
    try:
        if kind in ("agv", "rsv"):
            sizes = [int(v) * vec for v in rng.choice([0, 1, 3, 64, 1000, 5000], size=R)]
            if sum(sizes) == 0:
                sizes[0] = vec
            total = sum(sizes)
            x = gen.rank_inputs(R, total, dtype, seed=seed)
            if kind == "rsv":
                outs, _ = s.execute(s.build_v(sizes, chunk, coll=B.PL_REDUCE_SCATTERV, datapath=dp), x, repeats=2)
                ref = oracle.reduce_scatterv(x, sizes, dtype)
                for r in range(R):
                    assert outs[r].size == sizes[r] * es
                    if not sizes[r]:
                        continue
                    if dtype == "i32":
                        assert np.array_equal(outs[r].view(np.int32), ref[r])
                    elif dtype == "bf16":
                        check_float(gen.bf16_bits_to_f64(outs[r].view(np.uint16)), ref[r], dtype)
                    else:
                        check_float(outs[r].view(np.float32).astype(np.float64), ref[r], dtype)
            else:
                contrib = [x[p][: sizes[p]].copy() for p in range(R)]
                outs, _ = s.execute(s.build_v(sizes, chunk, coll=B.PL_ALLGATHERV, datapath=dp), contrib, repeats=2)
                ref = oracle.allgatherv(contrib)
                for r in range(R):
                    assert np.array_equal(outs[r], ref[r].view(np.uint8))
        elif kind == "a2av":
            counts = (rng.choice([0, 1, 2, 40, 700], size=(R, R)) * vec).astype(np.int64)
            x = [gen.rank_inputs(1, max(int(counts[p].sum()), vec), dtype, seed=seed * 31 + p)[0] for p in range(R)]
            outs, _ = s.execute(s.build_v(counts.reshape(-1).tolist(), chunk, datapath=dp), x, repeats=2)
            ref = oracle.alltoallv([a[: int(counts[p].sum())] for p, a in enumerate(x)], counts)
            for r in range(R):
                assert np.array_equal(outs[r][: ref[r].size * es], ref[r].view(np.uint8))
        else:
            root = int(rng.integers(0, R))
            m = int(rng.choice([1, 5, 300, 4099])) * vec
            n = R * m
            x = gen.rank_inputs(R, n, dtype, seed=seed)
            empty = np.zeros(0, x[0].dtype)
            coll = {"broadcast": B.PL_BROADCAST, "reduce": B.PL_REDUCE, "scatter": B.PL_SCATTER, "gather": B.PL_GATHER}[kind]
            count = n if kind in ("broadcast", "reduce") else m
            sched = B.pl_schedule_build_rooted(s.comm, coll, root, count, chunk, B.make_opts(datapath=dp))
            s.scheds.append(sched)
            if kind == "broadcast":
                outs, _ = s.execute(sched, [x[r] if r == root else empty for r in range(R)], repeats=2)
                for r in range(R):
                    assert np.array_equal(outs[r], x[root].view(np.uint8))
            elif kind == "reduce":
                outs, _ = s.execute(sched, x, repeats=2)
                ref = oracle.reduce(x, root, dtype)[root]
                if dtype == "i32":
                    assert np.array_equal(outs[root].view(np.int32), ref)
                elif dtype == "bf16":
                    check_float(gen.bf16_bits_to_f64(outs[root].view(np.uint16)), ref, dtype)
                else:
                    check_float(outs[root].view(np.float32).astype(np.float64), ref, dtype)
            elif kind == "scatter":
                outs, _ = s.execute(sched, [x[r] if r == root else empty for r in range(R)], repeats=2)
                ref = oracle.scatter(x, root)
                for r in range(R):
                    assert np.array_equal(outs[r], ref[r].view(np.uint8))
            else:
                contrib = [a[:m].copy() for a in x]
                outs, _ = s.execute(sched, contrib, repeats=2)
                assert np.array_equal(outs[root], oracle.gather(contrib, root)[root].view(np.uint8))
    finally:
        s.close()


@pytest.mark.parametrize("seed", range(60))
def test_random_hook_stage_ahead_and_packet_cases_match_the_oracle(seed):
    """Seeded draws over the options of the processing phase (scale, second operand, fp32 output),
    double-buffered staging (back-to-back executes with different inputs) and the packet datapath
    (layered one-shot all-reduce), with ragged sizes, odd rank counts, both executors."""
    import torch
    from gpu_harness import poison, stream_handle, to_dev
    rng = np.random.default_rng(9000 + seed)
    kind = str(rng.choice(["hook", "stage_ahead", "packets"]))
    R = int(rng.choice([2, 3, 4, 5, 7, 8, 12, 16]))
    vecs = int(rng.choice([1, 3, 17, 64, 257, 1031]))
    dp = int(rng.choice([B.PL_DP_AUTO, B.PL_DP_LDST, B.PL_DP_TMA]))

    def run(sched, ses, x, aux=None):
        info = B.pl_schedule_info(sched)
        d_in = [to_dev(a) for a in x]
        d_aux = [to_dev(a) for a in aux] if aux is not None else None
        d_out = [poison(info.out_bytes[r]) for r in range(R)]
        bufs = B.make_bufs([t.data_ptr() for t in d_in], [t.data_ptr() for t in d_out],
                           [int(info.in_bytes[r]) for r in range(R)], [int(info.out_bytes[r]) for r in range(R)],
                           [t.data_ptr() for t in d_aux] if d_aux else None,
                           [int(info.aux_bytes[r]) for r in range(R)] if d_aux else None)
        B.pl_execute(sched, bufs, stream_handle())
        return d_in, d_aux, d_out, info

    if kind == "hook":
        dtype = str(rng.choice(["bf16", "f32"]))
        es = B.DTYPE_SIZE[DT[dtype]]
        coll, algo = [(B.PL_REDUCE_SCATTER, B.PL_ALGO_DIRECT), (B.PL_REDUCE_SCATTER, B.PL_ALGO_RING),
                      (B.PL_ALLREDUCE, B.PL_ALGO_ONESHOT), (B.PL_ALLREDUCE, B.PL_ALGO_DIRECT_FUSED)][int(rng.integers(0, 4))]
        hook = int(rng.choice([1, 2, 3])) if dtype == "bf16" else 1
        scale = float(rng.choice([1.0, 0.5, 1.0 / R, -2.0]))
        n = R * vecs * (16 // es)
        n_out = n // R if coll == B.PL_REDUCE_SCATTER else n
        x = gen.rank_inputs(R, n, "f32n" if dtype == "f32" else dtype, seed=seed)
        aux = gen.rank_inputs(R, n_out, "f32n" if dtype == "f32" else dtype, seed=seed + 500) if hook & 1 else None
        ref = (oracle.allreduce_processed if coll == B.PL_ALLREDUCE else oracle.reduce_scatter_processed)(x, dtype, scale, aux)
        ses = Session(R, dtype)
        try:
            sched = ses.build(coll, algo, n, 16 * int(rng.choice([1, 5, 64, 3000])), datapath=dp, hook=hook, out_scale=scale,
                              slice_bytes=16 * int(rng.choice([0, 1, 128])))
            keep = run(sched, ses, x, aux)
            torch.cuda.synchronize()
            assert B.pl_comm_status(ses.comm).code == B.PL_OK
            d_out, info = keep[2], keep[3]
            for r in range(R):
                got = d_out[r][: int(info.out_bytes[r])].cpu().numpy()
                if hook & 2:
                    lo, hi = (r * n_out, (r + 1) * n_out) if coll == B.PL_REDUCE_SCATTER else (0, n)
                    mag = abs(scale) * sum(np.abs(gen.bf16_bits_to_f64(a[lo:hi])) for a in x)
                    if aux is not None:
                        mag = mag + np.abs(gen.bf16_bits_to_f64(aux[r]))
                    assert np.all(np.abs(got.view(np.float32).astype(np.float64) - ref[r]) <= (R + 1) * 2.0 ** -24 * mag + 1e-30)
                elif dtype == "bf16":
                    # the scale may enlarge the sum: the bf16 bound is relative to the processed value
                    check_float(gen.bf16_bits_to_f64(got.view(np.uint16)), ref[r], "bf16")
                else:
                    a64 = aux[r].astype(np.float64)
                    assert np.all(np.abs(got.view(np.float32).astype(np.float64) - ref[r]) <= 1e-6 * (np.abs(ref[r] - a64) + np.abs(a64)) + 1e-7)
        finally:
            ses.close()
    elif kind == "stage_ahead":
        dtype = str(rng.choice(["i32", "bf16"]))
        es = B.DTYPE_SIZE[DT[dtype]]
        coll = int(rng.choice([B.PL_ALLREDUCE, B.PL_REDUCE_SCATTER, B.PL_ALLGATHER, B.PL_ALLTOALL]))
        chunk_vecs = int(rng.choice([1, 5, 64, 512]))
        n = R * vecs * (16 // es)
        count = n // R if coll == B.PL_ALLGATHER else n
        cap = int(rng.choice([0, 2])) * 16 * min(chunk_vecs, vecs) * (1 if coll == B.PL_ALLGATHER else R)
        ses = Session(R, dtype)
        try:
            sched = ses.build(coll, B.PL_ALGO_DIRECT, count, 16 * chunk_vecs, datapath=dp, staging_bytes=cap,
                              flags=B.PL_OPT_STAGED | B.PL_OPT_OVERLAP_LAUNCH | B.PL_OPT_STAGE_AHEAD)
            calls, kept = 3, []
            xs = []
            for k in range(calls):
                x = gen.rank_inputs(R, n, dtype, seed=seed * 7 + k)
                if dtype == "i32":
                    x = [(a.astype(np.int64) * (k + 2) + k).astype(np.int32) for a in x]
                if coll == B.PL_ALLGATHER:
                    x = [a[:count].copy() for a in x]
                xs.append(x)
                kept.append(run(sched, ses, x))     # back to back, no synchronisation in between
            torch.cuda.synchronize()
            assert B.pl_comm_status(ses.comm).code == B.PL_OK
            for k in range(calls):
                x, (_, _, d_out, info) = xs[k], kept[k]
                ref = {B.PL_ALLREDUCE: lambda: oracle.allreduce(x, dtype), B.PL_REDUCE_SCATTER: lambda: oracle.reduce_scatter(x, dtype),
                       B.PL_ALLGATHER: lambda: oracle.allgather(x), B.PL_ALLTOALL: lambda: oracle.alltoall(x)}[coll]()
                for r in range(R):
                    got = d_out[r][: int(info.out_bytes[r])].cpu().numpy()
                    if coll in (B.PL_ALLGATHER, B.PL_ALLTOALL) or dtype == "i32":
                        assert np.array_equal(got, np.ascontiguousarray(ref[r]).view(np.uint8).reshape(-1)), (k, r)
                    else:
                        check_float(gen.bf16_bits_to_f64(got.view(np.uint16)), ref[r], "bf16")
        finally:
            ses.close()
    else:
        dtype = str(rng.choice(["i32", "bf16", "f32"]))
        es = B.DTYPE_SIZE[DT[dtype]]
        layers = int(rng.choice([1, 2, 5, 9]))
        vecs = min(vecs, 257)     # a CTA's threads hold at most 4 vectors each: 1024 per CTA
        n = vecs * (16 // es)
        ses = Session(R, dtype)
        try:
            g = int(rng.choice([0, 1, 2, 4, 8]))
            if g and vecs % g:
                g = 1
            sched = ses.build_layers(B.PL_ALGO_ONESHOT, n, layers, datapath=B.PL_DP_PACKET, n_ctas=g * R)
            for rep in range(2):
                x = [np.concatenate([gen.rank_inputs(R, n, "f32n" if dtype == "f32" else dtype, seed=seed * 13 + rep, stream_base=l * R)[r]
                                     for l in range(layers)]) for r in range(R)]
                if dtype == "i32":
                    x = [(a.astype(np.int64) * (rep + 1) + np.repeat(np.arange(layers), n) * 101).astype(np.int32) for a in x]
                outs, _ = ses.execute(sched, x)
                for l in range(layers):
                    ref = oracle.allreduce([a[l * n:(l + 1) * n] for a in x], dtype)
                    for r in range(R):
                        got = outs[r][l * n * es:(l + 1) * n * es]
                        if dtype == "i32":
                            assert np.array_equal(got.view(np.int32), ref[r])
                        elif dtype == "bf16":
                            check_float(gen.bf16_bits_to_f64(got.view(np.uint16)), ref[r], "bf16")
                        else:
                            check_float(got.view(np.float32).astype(np.float64), ref[r], "f32")
        finally:
            ses.close()


@pytest.mark.parametrize("seed", range(32))
def test_random_sm_window_and_l2_option_cases_match_the_oracle(seed):
    """Flag-free schedules of the bulk-copy datapath (direct reduce-scatter, all-gather, all-to-all)
    under random idle-SM windows and L2 options, odd rank counts and ragged sizes included: the
    grid must be every SM outside the window and a multiple of R."""
    import torch
    rng = np.random.default_rng(5000 + seed)
    sms = torch.cuda.get_device_properties(0).multi_processor_count
    R = int(rng.choice([2, 3, 4, 5, 7, 8, 12, 16]))
    dtype = str(rng.choice(["i32", "bf16", "f32"]))
    coll = int(rng.choice([B.PL_REDUCE_SCATTER, B.PL_ALLGATHER, B.PL_ALLTOALL]))
    es = B.DTYPE_SIZE[DT[dtype]]
    vecs = int(rng.choice([17, 257, 1031, 4099, 20011]))
    n = R * vecs * (16 // es)
    count = n // R if coll == B.PL_ALLGATHER else n
    # a window whose complement is a multiple of R
    active = int(rng.integers(max(1, (sms * 3 // 4) // R), sms // R + 1)) * R
    idle = sms - active
    flags = int(rng.choice([0, B.PL_OPT_INPUTS_LAST_USE, B.PL_OPT_NO_L2_HINTS]))
    kw = dict(datapath=B.PL_DP_TMA, flags=flags, slice_bytes=16 * int(rng.choice([0, 64, 1024])))
    if idle > 0:
        kw.update(idle_sm_first=int(rng.integers(0, sms - idle + 1)), idle_sm_count=idle)
    s = Session(R, dtype)
    try:
        sched = s.build(coll, B.PL_ALGO_DIRECT, count, 16 * int(rng.choice([64, 512, 1 << 20])), **kw)
        info = B.pl_schedule_info(sched)
        if idle > 0:
            assert (info.grid, info.idle_sm_count) == (active, idle)
        x = gen.rank_inputs(R, n, dtype, seed=seed)
        if coll == B.PL_ALLGATHER:
            x = [a[:count].copy() for a in x]
        outs, _ = s.execute(sched, x, repeats=3)
        if coll == B.PL_REDUCE_SCATTER:
            ref = oracle.reduce_scatter(x, dtype)
        elif coll == B.PL_ALLGATHER:
            ref = oracle.allgather(x)
        else:
            ref = oracle.alltoall(x)
        for r in range(R):
            if coll != B.PL_REDUCE_SCATTER or dtype == "i32":
                assert np.array_equal(outs[r], np.ascontiguousarray(ref[r]).view(np.uint8).reshape(-1)), (seed, r)
            elif dtype == "bf16":
                check_float(gen.bf16_bits_to_f64(outs[r].view(np.uint16)), ref[r], dtype)
            else:
                check_float(outs[r].view(np.float32).astype(np.float64), ref[r], dtype)
    finally:
        s.close()
