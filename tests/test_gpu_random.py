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
