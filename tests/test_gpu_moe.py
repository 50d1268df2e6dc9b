"""GPU parity of MoE dispatch / combine against the CPU oracle."""
import numpy as np
import pytest
import torch

from oracle import oracle
from paper_2609_36954_b200 import binding as B
from paper_2609_36954_b200 import inputs as gen

from gpu_harness import check_float, poison, stream_handle, to_dev

pytestmark = pytest.mark.gpu


class MoeRun:
    def __init__(self, R, T, H, E, K, cap, dtype=B.PL_BF16):
        self.R, self.T, self.H, self.E, self.K, self.cap = R, T, H, E, K, cap
        self.es = B.DTYPE_SIZE[dtype]
        self.comm = B.pl_comm_create(R, dtype)
        self.plan = B.pl_moe_plan_create(self.comm, T, H, E, K, cap)

    def dispatch(self, x, idx, with_meta=True):
        R = self.R
        self.d_x = [to_dev(a) for a in x]
        self.d_idx = [to_dev(a) for a in idx]
        self.d_recv = [poison(self.cap * self.H * self.es) for _ in range(R)]
        self.d_meta = [poison(self.cap * 16) for _ in range(R)] if with_meta else None
        B.pl_moe_dispatch(self.plan, [t.data_ptr() for t in self.d_x], [t.data_ptr() for t in self.d_idx],
                          [t.data_ptr() for t in self.d_recv],
                          [t.data_ptr() for t in self.d_meta] if with_meta else None, stream_handle())
        pos = np.zeros((R, self.T, self.K), np.int32)
        counts = np.zeros((R, R), np.int64)
        ecounts = np.zeros((R, self.E), np.int64)
        st = B.pl_moe_plan_read(self.plan, pos.ctypes.data, counts.ctypes.data, ecounts.ctypes.data, stream_handle())
        recv = [t.cpu().numpy() for t in self.d_recv]
        meta = [t.cpu().numpy().view(np.int32).reshape(-1, 4) for t in self.d_meta] if with_meta else None
        return st, recv, meta, pos, counts, ecounts

    def combine(self, y_dev, gates):
        R = self.R
        self.d_g = [to_dev(g) for g in gates]
        d_out = [poison(self.T * self.H * self.es) for _ in range(R)]
        B.pl_moe_combine(self.plan, [t.data_ptr() for t in y_dev], [t.data_ptr() for t in self.d_g],
                         [t.data_ptr() for t in d_out], stream_handle())
        torch.cuda.synchronize()
        return [t.cpu().numpy().view(np.uint16).reshape(self.T, self.H) for t in d_out]

    def close(self):
        B.pl_moe_plan_destroy(self.plan)
        B.pl_comm_destroy(self.comm)


@pytest.mark.parametrize("R,T,H,E,K,ident", [
    (8, 300, 1024, 64, 8, False),      # ragged token block (300 = 256 + 44)
    (4, 512, 7168, 32, 4, True),       # paper-like row width, hot experts on rank 0
    (2, 37, 8, 4, 2, False),           # tiny: 16-byte rows
    (8, 256, 16384, 256, 8, False),    # rows wider than one bulk-copy tile (2 tiles)
])
def test_dispatch_bit_exact_and_combine_within_tolerance(R, T, H, E, K, ident):
    idx, gates = gen.moe_routing(R, T, E, K, seed=0, identity_perm=ident)
    x = gen.moe_tokens_bf16(R, T, H, seed=2)
    cap = R * T * K if (ident or T < 64) else max(64, (R * T * K) // 2)
    ref = oracle.moe_dispatch(x, idx, E, recv_capacity_rows=cap)
    run = MoeRun(R, T, H, E, K, cap)
    try:
        for rep in range(2):
            st, recv, meta, pos, counts, ecounts = run.dispatch(x, idx)
            assert st == B.PL_OK
            assert np.array_equal(counts, ref["counts"])
            assert np.array_equal(ecounts, ref["expert_counts"])
            assert counts.sum() == R * T * K
            for p in range(R):
                assert np.array_equal(pos[p], ref["pos"][p])
            for r in range(R):
                nrows = int(counts[:, r].sum())
                got = recv[r].view(np.uint16).reshape(cap, H)[:nrows]
                assert np.array_equal(got, ref["recv"][r][:nrows]), f"recv rows of rank {r}"
                assert np.array_equal(meta[r][:nrows], ref["meta"][r][:nrows])
                # rows beyond the received ones are untouched (still poison)
                assert np.all(recv[r].reshape(cap, -1)[nrows:] == 0xFF)
        # combine with identity experts (y = what dispatch delivered)
        out = run.combine(run.d_recv, gates)
        want = oracle.moe_combine(ref["recv"], idx, ref["pos"], gates, E, H)
        for p in range(R):
            check_float(gen.bf16_bits_to_f64(out[p]), want[p], "bf16")
        # one-hot gates: an exact copy of the selected slot's row
        oh = [np.zeros((T, K), np.float32) for _ in range(R)]
        for g in oh:
            g[:, K - 1] = 1.0
        out = run.combine(run.d_recv, oh)
        for p in range(R):
            # equal as numbers: +0 + 1*(-0) is +0 in fp32, so a -0 input comes back as +0
            assert np.array_equal(gen.bf16_bits_to_f32(out[p]), gen.bf16_bits_to_f32(x[p]))
            assert np.array_equal(out[p][x[p] != 0x8000], x[p][x[p] != 0x8000])
    finally:
        run.close()


def test_combine_with_expert_dependent_rows():
    # y row = f(expert, source): checks that combine gathers the right row for every slot
    R, T, H, E, K = 4, 128, 256, 16, 4
    idx, gates = gen.moe_routing(R, T, E, K, seed=3)
    x = gen.moe_tokens_bf16(R, T, H, seed=5)
    cap = R * T * K
    ref = oracle.moe_dispatch(x, idx, E, recv_capacity_rows=cap)
    y = []
    for r in range(R):
        rows = gen.normal_bf16(cap * H, 77, r).reshape(cap, H)
        y.append(rows)
    run = MoeRun(R, T, H, E, K, cap)
    try:
        st, *_ = run.dispatch(x, idx, with_meta=False)
        assert st == B.PL_OK
        out = run.combine([to_dev(a) for a in y], gates)
        want = oracle.moe_combine(y, idx, ref["pos"], gates, E, H)
        for p in range(R):
            check_float(gen.bf16_bits_to_f64(out[p]), want[p], "bf16")
    finally:
        run.close()


def test_dispatch_int_rows_and_overflow_flag():
    R, T, E, K, W = 4, 64, 8, 2, 4
    idx, _ = gen.moe_routing(R, T, E, K, seed=6, identity_perm=True)
    x = [np.stack([np.full(W, p * 100000 + t, dtype=np.int32) for t in range(T)]) for p in range(R)]
    full = oracle.moe_dispatch(x, idx, E)
    need = int(full["counts"].sum(axis=0).max())
    run = MoeRun(R, T, W, E, K, need, dtype=B.PL_I32)
    try:
        st, recv, meta, pos, counts, _ = run.dispatch(x, idx)
        assert st == B.PL_OK
        for r in range(R):
            n = int(counts[:, r].sum())
            assert np.array_equal(recv[r].view(np.int32).reshape(need, W)[:n], full["recv"][r][:n])
    finally:
        run.close()
    run = MoeRun(R, T, W, E, K, need - 1, dtype=B.PL_I32)
    try:
        st, *_ = run.dispatch(x, idx)
        assert st == B.PL_ERR_OVERFLOW  # dropped rows are reported, nothing faults
    finally:
        run.close()


def test_moe_argument_errors():
    comm = B.pl_comm_create(4, B.PL_BF16)
    try:
        for args in [(16, 64, 6, 2, 100), (16, 4, 8, 2, 100), (16, 64, 8, 40, 100), (16, 64, 8, 2, 0)]:
            with pytest.raises(B.PurlinError):
                B.pl_moe_plan_create(comm, *args)
    finally:
        B.pl_comm_destroy(comm)


def test_moe_sixteen_ranks_topk_32():
    R, T, H, E, K = 16, 96, 64, 64, 32          # the widest top-k and communicator the plan accepts
    idx, gates = gen.moe_routing(R, T, E, K, seed=8)
    x = gen.moe_tokens_bf16(R, T, H, seed=9)
    cap = R * T * K
    ref = oracle.moe_dispatch(x, idx, E, recv_capacity_rows=cap)
    run = MoeRun(R, T, H, E, K, cap)
    try:
        st, recv, meta, pos, counts, ecounts = run.dispatch(x, idx)
        assert st == B.PL_OK and np.array_equal(counts, ref["counts"])
        for r in range(R):
            n = int(counts[:, r].sum())
            assert np.array_equal(recv[r].view(np.uint16).reshape(cap, H)[:n], ref["recv"][r][:n])
            assert np.array_equal(meta[r][:n], ref["meta"][r][:n])
        out = run.combine(run.d_recv, gates)
        want = oracle.moe_combine(ref["recv"], idx, ref["pos"], gates, E, H)
        for p in range(R):
            check_float(gen.bf16_bits_to_f64(out[p]), want[p], "bf16")
    finally:
        run.close()


# ---- deduplicated variant: one row per (token, destination rank) ------------------------------
@pytest.mark.parametrize("R,T,H,E,K,ident", [(8, 300, 512, 64, 8, False), (4, 700, 7168, 32, 4, True), (2, 40, 8, 8, 4, False)])
def test_dedup_dispatch_and_combine(R, T, H, E, K, ident):
    idx, _ = gen.moe_routing(R, T, E, K, seed=4, identity_perm=ident)
    x = gen.moe_tokens_bf16(R, T, H, seed=6)
    cap = R * T
    ref = oracle.moe_dispatch_dedup(x, idx, E, recv_capacity_rows=cap)
    run = MoeRun(R, T, H, E, K, cap)
    try:
        d_x = [to_dev(a) for a in x]
        d_i = [to_dev(a) for a in idx]
        for rep in range(2):
            d_recv = [poison(cap * H * 2) for _ in range(R)]
            d_meta = [poison(cap * 16) for _ in range(R)]
            B.pl_moe_dispatch_dedup(run.plan, [t.data_ptr() for t in d_x], [t.data_ptr() for t in d_i],
                                    [t.data_ptr() for t in d_recv], [t.data_ptr() for t in d_meta], stream_handle())
            pos = np.zeros((R, T, R), np.int32)
            counts = np.zeros((R, R), np.int64)
            assert B.pl_moe_plan_read_dedup(run.plan, pos.ctypes.data, counts.ctypes.data, stream_handle()) == B.PL_OK
            assert np.array_equal(counts, ref["counts"])
            for p in range(R):
                assert np.array_equal(pos[p], ref["pos"][p])
            for r in range(R):
                n = int(counts[:, r].sum())
                got = d_recv[r].cpu().numpy().view(np.uint16).reshape(cap, H)
                assert np.array_equal(got[:n], ref["recv"][r][:n])
                assert np.all(d_recv[r].cpu().numpy().reshape(cap, -1)[n:] == 0xFF)
                assert np.array_equal(d_meta[r].cpu().numpy().view(np.int32).reshape(cap, 4)[:n], ref["meta"][r][:n])
        # fewer rows cross than without deduplication
        assert counts.sum() <= R * T * K
        # combine: every destination returns one row per received row
        z = [gen.normal_bf16(cap * H, 90, r).reshape(cap, H) for r in range(R)]
        d_z = [to_dev(a) for a in z]
        d_out = [poison(T * H * 2) for _ in range(R)]
        B.pl_moe_combine_dedup(run.plan, [t.data_ptr() for t in d_z], [t.data_ptr() for t in d_out], stream_handle())
        torch.cuda.synchronize()
        want = oracle.moe_combine_dedup(z, ref["pos"], H)
        for p in range(R):
            got = gen.bf16_bits_to_f64(d_out[p].cpu().numpy().view(np.uint16).reshape(T, H))
            check_float(got, want[p], "bf16")
        # the plain dispatch on the same plan still works afterwards
        st, recv, *_ = run.dispatch(x, idx, with_meta=False)
        assert st == B.PL_OK or st == B.PL_ERR_OVERFLOW  # cap = R*T rows may be too small for K rows per token
    finally:
        run.close()


@pytest.mark.parametrize("K", [8, 6, 1, 32])
def test_combine_with_gates_from_logits(K):
    R, T, H, E = 4, 96, 256, 64
    idx, _ = gen.moe_routing(R, T, E, K, seed=14)
    x = gen.moe_tokens_bf16(R, T, H, seed=15)
    cap = R * T * K
    ref = oracle.moe_dispatch(x, idx, E, recv_capacity_rows=cap)
    logits = [gen.normal_f32(T * K, 33, p).reshape(T, K) * 3.0 for p in range(R)]
    # reference gates: softmax in fp64, handed to the oracle as the fp32 values nearest to them
    gates64 = [np.exp(l.astype(np.float64) - l.astype(np.float64).max(axis=1, keepdims=True)) for l in logits]
    gates = [np.ascontiguousarray((g / g.sum(axis=1, keepdims=True)).astype(np.float32)) for g in gates64]
    y = [gen.normal_bf16(cap * H, 77, r).reshape(cap, H) for r in range(R)]
    want = oracle.moe_combine(y, idx, ref["pos"], gates, E, H)
    run = MoeRun(R, T, H, E, K, cap)
    try:
        st, *_ = run.dispatch(x, idx, with_meta=False)
        assert st == B.PL_OK
        d_y = [to_dev(a) for a in y]
        d_l = [to_dev(a) for a in logits]
        d_out = [poison(T * H * 2) for _ in range(R)]
        B.pl_moe_combine_logits(run.plan, [t.data_ptr() for t in d_y], [t.data_ptr() for t in d_l],
                                [t.data_ptr() for t in d_out], stream_handle())
        torch.cuda.synchronize()
        for p in range(R):
            got = gen.bf16_bits_to_f64(d_out[p].cpu().numpy().view(np.uint16).reshape(T, H))
            check_float(got, want[p], "bf16")
    finally:
        run.close()


@pytest.mark.parametrize("seed", range(24))
def test_random_moe_shapes_match_the_oracle(seed):
    """Seeded draws of rank count, tokens, row width, expert count and top-k, including one
    token per rank, experts that nobody selects and rows of a single 16-byte vector."""
    rng = np.random.default_rng(500 + seed)
    R = int(rng.choice([2, 3, 4, 8, 16]))
    epr = int(rng.choice([1, 2, 5, 32]))
    E = R * epr
    K = int(rng.choice([k for k in (1, 2, 4, 8, 32) if k <= E]))
    T = int(rng.choice([1, 2, 31, 256, 257, 600]))
    H = int(rng.choice([8, 24, 512, 1000, 7168]))
    ident = bool(rng.integers(0, 2))
    idx, gates = gen.moe_routing(R, T, E, K, seed=seed, identity_perm=ident)
    x = gen.moe_tokens_bf16(R, T, H, seed=seed + 1)
    cap = R * T * K
    ref = oracle.moe_dispatch(x, idx, E, recv_capacity_rows=cap)
    run = MoeRun(R, T, H, E, K, cap)
    try:
        st, recv, meta, pos, counts, ecounts = run.dispatch(x, idx)
        assert st == B.PL_OK
        assert np.array_equal(counts, ref["counts"]) and np.array_equal(ecounts, ref["expert_counts"])
        for p in range(R):
            assert np.array_equal(pos[p], ref["pos"][p])
        for r in range(R):
            nrows = int(counts[:, r].sum())
            assert np.array_equal(recv[r].view(np.uint16).reshape(cap, H)[:nrows], ref["recv"][r][:nrows])
            assert np.array_equal(meta[r][:nrows], ref["meta"][r][:nrows])
            assert np.all(recv[r].reshape(cap, -1)[nrows:] == 0xFF)
        out = run.combine(run.d_recv, gates)
        want = oracle.moe_combine(ref["recv"], idx, ref["pos"], gates, E, H)
        for p in range(R):
            check_float(gen.bf16_bits_to_f64(out[p]), want[p], "bf16")
    finally:
        run.close()


def test_a_second_smaller_plan_does_not_break_the_first():
    """The kernels' shared-memory limit is a property of the function, not of a plan: a plan with
    wide rows (86 KiB of tiles per CTA, above the 48 KiB default) must keep working after a plan
    with narrow rows and few experts has been created."""
    R, T, H, E, K = 4, 96, 7168, 64, 4
    idx, gates = gen.moe_routing(R, T, E, K, seed=4)
    x = gen.moe_tokens_bf16(R, T, H, seed=6)
    cap = R * T * K
    ref = oracle.moe_dispatch(x, idx, E, recv_capacity_rows=cap)
    big = MoeRun(R, T, H, E, K, cap)
    small = MoeRun(2, 16, 256, 4, 2, 64)
    try:
        xs = gen.moe_tokens_bf16(2, 16, 256, seed=7)
        idxs, _ = gen.moe_routing(2, 16, 4, 2, seed=8)
        st, recv_s, _, _, counts_s, _ = small.dispatch(xs, idxs)
        refs = oracle.moe_dispatch(xs, idxs, 4, recv_capacity_rows=64)
        assert st == B.PL_OK and np.array_equal(counts_s, refs["counts"])
        st, recv, meta, pos, counts, ecounts = big.dispatch(x, idx)
        assert st == B.PL_OK
        assert np.array_equal(counts, ref["counts"])
        for r in range(R):
            nrows = int(counts[:, r].sum())
            assert np.array_equal(recv[r].view(np.uint16).reshape(cap, H)[:nrows], ref["recv"][r][:nrows])
    finally:
        small.close()
        big.close()
