"""GPU parity of the processing phase (Sec. 3.3: configurable while the sum sits in registers):
scale, second operand (residual), unconverted fp32 output, on both executors, against the oracle."""
import numpy as np
import pytest
import torch

from oracle import oracle
from paper_2609_36954_b200 import binding as B
from paper_2609_36954_b200 import inputs as gen

from gpu_harness import DT, Session, check_float, poison, stream_handle, to_dev

pytestmark = pytest.mark.gpu

DATAPATHS = [B.PL_DP_LDST, B.PL_DP_TMA]
CASES = [("rs_direct", B.PL_REDUCE_SCATTER, B.PL_ALGO_DIRECT), ("rs_ring", B.PL_REDUCE_SCATTER, B.PL_ALGO_RING),
         ("ar_oneshot", B.PL_ALLREDUCE, B.PL_ALGO_ONESHOT), ("ar_fused", B.PL_ALLREDUCE, B.PL_ALGO_DIRECT_FUSED)]


def run_hooked(ses, sched, x, aux):
    info = B.pl_schedule_info(sched)
    R = ses.R
    d_in = [to_dev(a) for a in x]
    d_aux = [to_dev(a) for a in aux] if aux is not None else None
    d_out = [poison(info.out_bytes[r]) for r in range(R)]
    bufs = B.make_bufs([t.data_ptr() for t in d_in], [t.data_ptr() for t in d_out],
                       [int(info.in_bytes[r]) for r in range(R)], [int(info.out_bytes[r]) for r in range(R)],
                       [t.data_ptr() for t in d_aux] if d_aux else None,
                       [int(info.aux_bytes[r]) for r in range(R)] if d_aux else None)
    for _ in range(2):
        B.pl_execute(sched, bufs, stream_handle())
    torch.cuda.synchronize()
    assert B.pl_comm_status(ses.comm).code == B.PL_OK
    return [d_out[r][: int(info.out_bytes[r])].cpu().numpy() for r in range(R)], info


def f32_out_tolerance(x, aux, scale, R):
    """fp32 image of scale * sum + aux: R - 1 additions, one multiplication and one more addition,
    each rounded to fp32 once (relative 2^-24 of a partial result that never exceeds the sum of
    magnitudes)."""
    mag = abs(scale) * sum(np.abs(gen.bf16_bits_to_f64(a)) for a in x)
    if aux is not None:
        mag = mag + np.abs(gen.bf16_bits_to_f64(aux))
    return (R + 1) * 2.0 ** -24 * mag + 1e-30


@pytest.mark.parametrize("dp", DATAPATHS)
@pytest.mark.parametrize("name,coll,algo", CASES)
@pytest.mark.parametrize("dtype,hook", [("bf16", B.PL_HOOK_RESIDUAL), ("bf16", B.PL_HOOK_F32_OUT),
                                        ("bf16", B.PL_HOOK_RESIDUAL | B.PL_HOOK_F32_OUT), ("f32", B.PL_HOOK_RESIDUAL)])
def test_processing_phase_matches_the_oracle(dp, name, coll, algo, dtype, hook):
    R = 8
    es = B.DTYPE_SIZE[DT[dtype]]
    part = 37 * 1024 + 16                       # ragged against tiles and slices
    n = R * part // es
    n_out = n // R if coll == B.PL_REDUCE_SCATTER else n
    scale = 0.375
    x = gen.rank_inputs(R, n, "f32n" if dtype == "f32" else dtype, seed=70)
    aux = gen.rank_inputs(R, n_out, "f32n" if dtype == "f32" else dtype, seed=71) if hook & B.PL_HOOK_RESIDUAL else None
    ref = (oracle.allreduce_processed if coll == B.PL_ALLREDUCE else oracle.reduce_scatter_processed)(x, dtype, scale, aux)
    ses = Session(R, dtype)
    try:
        s = ses.build(coll, algo, n, 16384, datapath=dp, hook=hook, out_scale=scale)
        outs, info = run_hooked(ses, s, x, aux)
        assert info.datapath == dp
        for r in range(R):
            if hook & B.PL_HOOK_F32_OUT:
                got = outs[r].view(np.float32).astype(np.float64)
                lo, hi = (r * n_out, (r + 1) * n_out) if coll == B.PL_REDUCE_SCATTER else (0, n)
                tol = f32_out_tolerance([a[lo:hi] for a in x], aux[r] if aux is not None else None, scale, R)
                assert np.all(np.abs(got - ref[r]) <= tol)
            elif dtype == "bf16":
                check_float(gen.bf16_bits_to_f64(outs[r].view(np.uint16)), ref[r], "bf16")
            else:
                # fp32 data: the sum itself carries the usual 1e-6 |sum| + 1e-7; the scaling and the
                # addition of the second operand each round once more, relative to their OPERANDS
                # (the result can cancel), so the bound is taken on |scale * sum| + |aux|
                got = outs[r].view(np.float32).astype(np.float64)
                operands = np.abs(ref[r] - aux[r].astype(np.float64)) + np.abs(aux[r].astype(np.float64))
                assert np.all(np.abs(got - ref[r]) <= 1e-6 * operands + 1e-7)
    finally:
        ses.close()


@pytest.mark.parametrize("dp", DATAPATHS)
def test_processing_phase_exact_cases(dp):
    """residual = -sum gives exactly zero; fp32 output of equal inputs is R * x bit for bit."""
    R, n = 8, 8 * 4096
    ints = [gen.f32_to_bf16_bits(((np.arange(n) % 7) - 3 + r).astype(np.float32)) for r in range(R)]
    exact = sum(gen.bf16_bits_to_f64(a) for a in ints)
    ses = Session(R, "bf16")
    try:
        for coll, algo in ((B.PL_ALLREDUCE, B.PL_ALGO_DIRECT_FUSED), (B.PL_REDUCE_SCATTER, B.PL_ALGO_RING)):
            m = n if coll == B.PL_ALLREDUCE else n // R
            aux = [gen.f32_to_bf16_bits((-exact[(0 if coll == B.PL_ALLREDUCE else r * m):][:m]).astype(np.float32)) for r in range(R)]
            s = ses.build(coll, algo, n, 8192, datapath=dp, hook=B.PL_HOOK_RESIDUAL)
            outs, _ = run_hooked(ses, s, ints, aux)
            for r in range(R):
                assert not np.any(outs[r].view(np.uint16) & 0x7FFF)      # +0 or -0 everywhere
        x = gen.normal_bf16(n, 3, 0)
        same = [x.copy() for _ in range(R)]
        s = ses.build(B.PL_ALLREDUCE, B.PL_ALGO_ONESHOT, n, 8192, datapath=dp, hook=B.PL_HOOK_F32_OUT)
        outs, _ = run_hooked(ses, s, same, None)
        want = (R * gen.bf16_bits_to_f64(x)).astype(np.float32)
        for r in range(R):
            assert np.array_equal(outs[r].view(np.float32), want)
    finally:
        ses.close()


def test_layered_fused_allreduce_with_residual():
    """The decode shape with the residual connection folded into the all-reduce, 6 layers per launch."""
    R, n, layers = 8, 8192, 6
    x = [np.concatenate([gen.normal_bf16(n, 0, l * R + r) for l in range(layers)]) for r in range(R)]
    aux = [np.concatenate([gen.normal_bf16(n, 1, l * R + r) for l in range(layers)]) for r in range(R)]
    ses = Session(R, "bf16")
    try:
        s = ses.build_layers(B.PL_ALGO_DIRECT_FUSED, n, layers, hook=B.PL_HOOK_RESIDUAL)
        outs, _ = run_hooked(ses, s, x, aux)
        for l in range(layers):
            sl = slice(l * n, (l + 1) * n)
            ref = oracle.allreduce_processed([a[sl] for a in x], "bf16", 1.0, [a[sl] for a in aux])
            for r in range(R):
                check_float(gen.bf16_bits_to_f64(outs[r].view(np.uint16)[sl]), ref[r], "bf16")
    finally:
        ses.close()


def test_hooked_execute_needs_the_second_operand():
    R, n = 4, 4 * 1024
    ses = Session(R, "bf16")
    try:
        s = ses.build(B.PL_REDUCE_SCATTER, B.PL_ALGO_DIRECT, n, 4096, hook=B.PL_HOOK_RESIDUAL)
        info = B.pl_schedule_info(s)
        d_in = [poison(info.in_bytes[r]) for r in range(R)]
        d_out = [poison(info.out_bytes[r]) for r in range(R)]
        ins, outs = [t.data_ptr() for t in d_in], [t.data_ptr() for t in d_out]
        ib, ob = [int(info.in_bytes[r]) for r in range(R)], [int(info.out_bytes[r]) for r in range(R)]
        with pytest.raises(B.PurlinError) as e:          # no aux at all
            B.pl_execute(s, B.make_bufs(ins, outs, ib, ob), stream_handle())
        assert e.value.status == B.PL_ERR_INVALID_ARG
        with pytest.raises(B.PurlinError) as e:          # aux overlapping an output
            B.pl_execute(s, B.make_bufs(ins, outs, ib, ob, outs, ob), stream_handle())
        assert e.value.status == B.PL_ERR_INVALID_ARG
        d_aux = [poison(info.aux_bytes[r] + 16) for r in range(R)]
        with pytest.raises(B.PurlinError) as e:          # misaligned aux
            B.pl_execute(s, B.make_bufs(ins, outs, ib, ob, [t.data_ptr() + 2 for t in d_aux], ob), stream_handle())
        assert e.value.status == B.PL_ERR_ALIGNMENT
    finally:
        ses.close()


@pytest.mark.parametrize("R", [3, 16])
@pytest.mark.parametrize("hook", [B.PL_HOOK_RESIDUAL, B.PL_HOOK_F32_OUT])
def test_hooked_fused_allreduce_on_the_bulk_copy_executor_at_other_rank_counts(R, hook):
    """The results of a hooked fused all-reduce leave through the ring slot (one operand / result
    tile per rank, or one wide result region): 16 ranks fill all 32 producer lanes, 3 ranks leave
    odd tile counts; sizes ragged against the stage capacity."""
    part = 21 * 1024 + 32
    n = R * part // 2
    scale = 0.5
    x = gen.rank_inputs(R, n, "bf16", seed=80 + R)
    aux = gen.rank_inputs(R, n, "bf16", seed=81 + R) if hook & B.PL_HOOK_RESIDUAL else None
    ref = oracle.allreduce_processed(x, "bf16", scale, aux)
    ses = Session(R, "bf16")
    try:
        s = ses.build(B.PL_ALLREDUCE, B.PL_ALGO_DIRECT_FUSED, n, 8192, datapath=B.PL_DP_TMA, hook=hook, out_scale=scale)
        outs, info = run_hooked(ses, s, x, aux)
        assert info.datapath == B.PL_DP_TMA
        for r in range(R):
            if hook & B.PL_HOOK_F32_OUT:
                got = outs[r].view(np.float32).astype(np.float64)
                assert np.all(np.abs(got - ref[r]) <= f32_out_tolerance(x, None, scale, R))
            else:
                check_float(gen.bf16_bits_to_f64(outs[r].view(np.uint16)), ref[r], "bf16")
    finally:
        ses.close()
