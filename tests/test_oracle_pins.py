"""Pins for the CPU oracle: closed forms, identities, special cases and brute force.

None of these re-types the oracle's own loop: each checks it against something the
mathematics fixes (rank-coded closed forms, numpy library routines on a stacked
[R][n] array, exactly rounded sums, involution / composition identities).
"""
import math

import numpy as np
import pytest

from oracle import oracle
from paper_2609_36954_b200 import inputs
from paper_2609_36954_b200 import inputs as gen


# ----------------------------------------------------------------------------- #
# integer closed forms (rank-coded inputs x_p[j] = p*n + j)
# ----------------------------------------------------------------------------- #
def test_allreduce_int_closed_form_config1():
    R, n = 4, 262144
    x = inputs.rank_coded_i32(R, n)
    out = oracle.allreduce(x, "i32")
    i = np.arange(n, dtype=np.int64)
    want = 4 * i + 1572864  # 4i + n*(0+1+2+3)
    for r in range(R):
        assert np.array_equal(out[r].astype(np.int64), want)


@pytest.mark.parametrize("R,m", [(2, 8), (3, 20), (5, 12), (8, 64)])
def test_reduce_scatter_int_closed_form(R, m):
    n = R * m
    x = inputs.rank_coded_i32(R, n)
    out = oracle.reduce_scatter(x, "i32")
    i = np.arange(m, dtype=np.int64)
    for r in range(R):
        want = R * (r * m + i) + n * R * (R - 1) // 2
        assert np.array_equal(out[r].astype(np.int64), want)


def test_int32_wraps():
    x = [np.array([2 ** 31 - 1, -5], dtype=np.int32), np.array([1, -(2 ** 31)], dtype=np.int32)]
    out = oracle.allreduce(x, "i32")
    assert out[0].tolist() == [-(2 ** 31), 2 ** 31 - 5]


# ----------------------------------------------------------------------------- #
# copy-only collectives against numpy routines on the stacked array
# ----------------------------------------------------------------------------- #
@pytest.mark.parametrize("R,m", [(2, 16), (3, 48), (8, 1000)])
def test_allgather_is_concatenation(R, m):
    x = inputs.rank_coded_bytes(R, m)
    out = oracle.allgather(x)
    want = np.concatenate(x)
    for r in range(R):
        assert np.array_equal(out[r], want)
    # spot value: out_r[p*m+i] is the byte rank p generated at position i
    p, i = R - 1, m // 2
    assert out[0][p * m + i] == int(inputs.hash_counter(0x5EED, p, np.uint64(i)) & np.uint64(0xFF))


@pytest.mark.parametrize("R,m", [(2, 16), (3, 48), (5, 7), (8, 256)])
def test_alltoall_is_block_transpose_and_involution(R, m):
    x = inputs.rank_coded_bytes(R, R * m)
    out = oracle.alltoall(x)
    stacked = np.stack(x).reshape(R, R, m)          # [p][r][i]
    want = stacked.transpose(1, 0, 2).reshape(R, R * m)  # [r][p][i]
    for r in range(R):
        assert np.array_equal(out[r], want[r])
    back = oracle.alltoall(out)
    for r in range(R):
        assert np.array_equal(back[r], x[r])


def _a2av_bruteforce(x, C):
    R = len(x)
    outs = []
    for r in range(R):
        pieces = []
        for p in range(R):
            lst = x[p].tolist()
            start = sum(int(C[p][q]) for q in range(r))
            pieces.extend(lst[start:start + int(C[p][r])])
        outs.append(pieces)
    return outs


def test_alltoallv_bruteforce_and_conservation():
    rng = np.random.default_rng(0)
    for R in (2, 3, 5):
        C = rng.integers(0, 9, size=(R, R))
        C[0, R - 1] = 0  # an empty segment
        x = [(np.arange(C[p].sum()) + 1000 * p).astype(np.int32) for p in range(R)]
        out = oracle.alltoallv(x, C)
        want = _a2av_bruteforce(x, C)
        for r in range(R):
            assert out[r].size == C[:, r].sum()
            assert out[r].tolist() == want[r]
        assert sum(o.size for o in out) == sum(a.size for a in x)


def test_alltoallv_uniform_counts_reduce_to_alltoall():
    R, m = 4, 24
    x = [inputs.uniform_f32(R * m, 7, r) for r in range(R)]
    a = oracle.alltoallv(x, np.full((R, R), m))
    b = oracle.alltoall(x)
    for r in range(R):
        assert np.array_equal(a[r], b[r])


def test_alltoallv_with_paper_zipf_counts():
    T = 8192
    C = inputs.alltoallv_counts_bytes(T)
    x = inputs.rank_coded_bytes(8, T)
    out = oracle.alltoallv(x, C)
    # receiver r's segment from source p starts after everything from lower sources
    r, p = 5, 3
    roff = int(C[:p, r].sum()); soff = int(C[p, :r].sum()); n = int(C[p, r])
    assert np.array_equal(out[r][roff:roff + n], x[p][soff:soff + n])
    assert all(o.size == T for o in out)


# ----------------------------------------------------------------------------- #
# reductions: composition identity, exact special cases, exactly-rounded sums
# ----------------------------------------------------------------------------- #
@pytest.mark.parametrize("dtype", ["bf16", "f32"])
def test_allreduce_equals_allgather_of_reduce_scatter(dtype):
    R, n = 8, 8 * 40
    x = inputs.rank_inputs(R, n, dtype, seed=3)
    ar = oracle.allreduce(x, dtype)
    rs = oracle.reduce_scatter(x, dtype)
    ag = oracle.allgather(rs)
    for r in range(R):
        assert np.array_equal(ar[r], ag[r])
    xi = inputs.rank_coded_i32(R, n)
    ari = oracle.allreduce(xi, "i32")
    agi = oracle.allgather(oracle.reduce_scatter(xi, "i32"))
    for r in range(R):
        assert np.array_equal(ari[r], agi[r])


def test_float_special_cases():
    R, n = 8, 64
    base = inputs.normal_bf16(n, 11, 0)
    f = inputs.bf16_bits_to_f64(base)
    # all ranks equal: R*x exactly (R a power of two)
    out = oracle.allreduce([base.copy() for _ in range(R)], "bf16")
    assert np.array_equal(out[3], R * f)
    # x_p = -x_{p+1} pairs cancel to exactly zero
    neg = base ^ np.uint16(0x8000)
    out = oracle.allreduce([base if p % 2 == 0 else neg for p in range(R)], "bf16")
    assert np.all(out[0] == 0.0)
    # a single non-zero rank: the sum is that rank's data
    zero = np.zeros(n, dtype=np.uint16)
    out = oracle.allreduce([base if p == 5 else zero for p in range(R)], "bf16")
    assert np.array_equal(out[7], f)
    # reduce-scatter picks partition r
    out = oracle.reduce_scatter([base if p == 2 else zero for p in range(R)], "bf16")
    m = n // R
    for r in range(R):
        assert np.array_equal(out[r], f[r * m:(r + 1) * m])


@pytest.mark.parametrize("dtype", ["bf16", "f32", "f32n"])
def test_float_sum_against_exactly_rounded_sum(dtype):
    R, n = 8, 96
    x = inputs.rank_inputs(R, n, dtype, seed=5)
    od = "bf16" if dtype == "bf16" else "f32"
    out = oracle.allreduce(x, od)
    as64 = [inputs.bf16_bits_to_f64(a) if dtype == "bf16" else a.astype(np.float64) for a in x]
    for i in range(n):
        exact = math.fsum(float(a[i]) for a in as64)
        # 8 bf16/fp32 addends in fp64: the running sum is exact or within 1 ulp
        assert abs(out[0][i] - exact) <= 2.0 ** -50 * max(1.0, abs(exact))
    # order sensitivity pin: the oracle adds rank 0 first (1e17 + 1 - 1e17 = 0 in fp64)
    a = [np.array([1e17], np.float32), np.array([1.0], np.float32), np.array([-1e17], np.float32)]
    got = oracle.allreduce(a, "f32")[0][0]
    big = float(np.float32(1e17))
    assert got == (big + 1.0) - big


def test_reduce_scatter_bruteforce_tiny():
    for R in (2, 3, 4, 5, 8):
        for mult in (1, 7):
            n = R * 8 * mult
            x = inputs.rank_inputs(R, n, "f32", seed=R)
            stacked = np.stack(x).astype(np.float64)  # [R][n]
            full = stacked.sum(axis=0)
            rs = oracle.reduce_scatter(x, "f32")
            ar = oracle.allreduce(x, "f32")
            m = n // R
            for r in range(R):
                assert np.allclose(rs[r], full[r * m:(r + 1) * m], rtol=0, atol=1e-15)
                assert np.allclose(ar[r], full, rtol=0, atol=1e-15)


# ----------------------------------------------------------------------------- #
# MoE dispatch / combine
# ----------------------------------------------------------------------------- #
def _row_coded_tokens(R, T, W=4):
    return [np.stack([np.full(W, p * 100000 + t, dtype=np.int32) for t in range(T)]) for p in range(R)]


def test_moe_dispatch_rows_meta_counts():
    R, T, E, K = 4, 64, 16, 4
    idx, _ = inputs.moe_routing(R, T, E, K, seed=9)
    x = _row_coded_tokens(R, T)
    d = oracle.moe_dispatch(x, idx, E)
    epr = E // R
    allidx = np.stack(idx)  # [R][T][K]
    assert d["counts"].sum() == R * T * K
    for p in range(R):
        assert np.array_equal(d["expert_counts"][p], np.bincount(idx[p].ravel(), minlength=E))
    for r in range(R):
        nrows = int(d["counts"][:, r].sum())
        meta = d["meta"][r][:nrows]
        # rows carry the token they claim to carry
        assert np.array_equal(d["recv"][r][:nrows, 0], meta[:, 0] * 100000 + meta[:, 1])
        # meta is consistent with the routing table and the expert placement
        assert np.array_equal(allidx[meta[:, 0], meta[:, 1], meta[:, 2]], meta[:, 3])
        assert np.all(meta[:, 3] // epr == r)
        # order: (source rank, expert, token) lexicographic, strictly increasing
        key = (meta[:, 0].astype(np.int64) * E + meta[:, 3]) * T + meta[:, 1]
        assert np.all(np.diff(key) > 0)
        assert np.all(d["meta"][r][nrows:] == -1)
    # pos is the inverse map
    for p in range(R):
        for t in (0, T // 2, T - 1):
            for j in range(K):
                r = idx[p][t, j] // epr
                assert d["meta"][r][d["pos"][p][t, j]].tolist() == [p, t, j, idx[p][t, j]]


def test_moe_dispatch_independent_lexsort_formulation():
    R, T, E, K = 3, 40, 6, 2
    idx, _ = inputs.moe_routing(R, T, E, K, seed=4)
    x = _row_coded_tokens(R, T, W=2)
    d = oracle.moe_dispatch(x, idx, E)
    epr = E // R
    for r in range(R):
        rows = []
        for p in range(R):
            tt, jj = np.nonzero(idx[p] // epr == r)
            ee = idx[p][tt, jj]
            order = np.lexsort((tt, ee))  # by expert, then token
            rows.append(x[p][tt[order]])
        want = np.concatenate(rows) if rows else np.zeros((0, 2), np.int32)
        assert np.array_equal(d["recv"][r][: want.shape[0]], want)


def test_moe_dispatch_k1_sorted_degenerates_to_alltoallv():
    R, T, E = 4, 32, 8
    rng = np.random.default_rng(1)
    idx = [np.sort(rng.integers(0, E, size=T)).astype(np.int32).reshape(T, 1) for _ in range(R)]
    x = _row_coded_tokens(R, T, W=4)
    d = oracle.moe_dispatch(x, idx, E)
    C = d["counts"]
    flat = [a.reshape(-1) for a in x]
    a2av = oracle.alltoallv(flat, C * 4)
    for r in range(R):
        n = int(C[:, r].sum())
        assert np.array_equal(d["recv"][r][:n].reshape(-1), a2av[r])


def test_moe_dispatch_capacity_overflow_reported():
    R, T, E, K = 2, 8, 4, 2
    idx, _ = inputs.moe_routing(R, T, E, K)
    with pytest.raises(RuntimeError):
        oracle.moe_dispatch(_row_coded_tokens(R, T), idx, E, recv_capacity_rows=3)


def test_moe_combine_identity_constant_and_onehot():
    R, T, E, K, H = 4, 32, 16, 4, 24
    idx, gates = inputs.moe_routing(R, T, E, K, seed=2)
    x = inputs.moe_tokens_bf16(R, T, H, seed=2)
    d = oracle.moe_dispatch(x, idx, E)
    # identity experts: combine returns sum_j g_j * x = x (gates sum to 1 up to fp32 rounding)
    out = oracle.moe_combine(d["recv"], idx, d["pos"], gates, E, H)
    for p in range(R):
        xf = inputs.bf16_bits_to_f64(x[p])
        assert np.all(np.abs(out[p] - xf) <= 2.0 ** -20 * np.abs(xf) + 1e-12)
    # expert-constant rows c_e = e + 1: out[t,:] = sum_j g[t,j] * (e_j + 1), from routing alone
    y = []
    for r in range(R):
        rows = np.zeros_like(d["recv"][r])
        n = int(d["counts"][:, r].sum())
        vals = (d["meta"][r][:n, 3] + 1).astype(np.float32)
        rows[:n] = inputs.f32_to_bf16_bits(vals)[:, None]
        y.append(rows)
    out = oracle.moe_combine(y, idx, d["pos"], gates, E, H)
    for p in range(R):
        want = (gates[p].astype(np.float64) * (idx[p] + 1)).sum(axis=1)
        assert np.allclose(out[p], want[:, None], rtol=1e-14, atol=0)
    # one-hot gates on slot 2: an exact copy of the slot-2 row
    oh = [np.zeros((T, K), np.float32) for _ in range(R)]
    for g in oh:
        g[:, 2] = 1.0
    out = oracle.moe_combine(d["recv"], idx, d["pos"], oh, E, H)
    for p in range(R):
        assert np.array_equal(out[p], inputs.bf16_bits_to_f64(x[p]))
    # gate weighting is per slot, not per row: a slot-dependent gate with slot-coded rows
    g2 = [np.tile(np.array([0.5, 0.25, 0.125, 0.125], np.float32), (T, 1)) for _ in range(R)]
    y2 = []
    for r in range(R):
        rows = np.zeros_like(d["recv"][r])
        n = int(d["counts"][:, r].sum())
        rows[:n] = inputs.f32_to_bf16_bits((d["meta"][r][:n, 2] + 1).astype(np.float32))[:, None]
        y2.append(rows)
    out = oracle.moe_combine(y2, idx, d["pos"], g2, E, H)
    assert np.all(out[0] == 0.5 * 1 + 0.25 * 2 + 0.125 * 3 + 0.125 * 4)


# ----------------------------------------------------------------------------- #
# V variants of all-gather and reduce-scatter
# ----------------------------------------------------------------------------- #
def test_allgatherv_is_ragged_concatenation():
    sizes = [5, 0, 12, 1, 7]
    x = [(np.arange(n) + 100 * p).astype(np.int32) for p, n in enumerate(sizes)]
    out = oracle.allgatherv(x)
    want = np.concatenate(x)
    for r in range(len(sizes)):
        assert np.array_equal(out[r], want)
    # equal sizes reduce to the fixed-size collective
    y = inputs.rank_coded_bytes(4, 48)
    a, b = oracle.allgatherv(y), oracle.allgather(y)
    for r in range(4):
        assert np.array_equal(a[r], b[r])


def test_reduce_scatterv_closed_form_uniform_case_and_zipf_sizes():
    R = 8
    sizes_bytes = inputs.zipf_split(8192)                 # the paper's split: 128-byte units 9 9 8 8 8 8 7 7
    sizes = (sizes_bytes // 4).tolist()
    n = sum(sizes)
    x = inputs.rank_coded_i32(R, n)                       # x_p[j] = p*n + j
    out = oracle.reduce_scatterv(x, sizes, "i32")
    off = 0
    for k in range(R):
        i = np.arange(sizes[k], dtype=np.int64)
        assert np.array_equal(out[k].astype(np.int64), R * (off + i) + n * R * (R - 1) // 2)
        off += sizes[k]
    # uniform sizes: identical to reduce-scatter; a zero-size partition yields an empty output
    xf = inputs.rank_inputs(4, 4 * 24, "bf16", seed=8)
    a, b = oracle.reduce_scatterv(xf, [24] * 4, "bf16"), oracle.reduce_scatter(xf, "bf16")
    for r in range(4):
        assert np.array_equal(a[r], b[r])
    c = oracle.reduce_scatterv(xf, [40, 0, 32, 24], "bf16")
    full = oracle.allreduce(xf, "bf16")[0]
    assert c[1].size == 0 and np.array_equal(c[2], full[40:72]) and np.array_equal(c[3], full[72:96])
    # gathering what the V reduce-scatter scattered rebuilds the all-reduce (paper's composition identity)
    assert np.array_equal(np.concatenate(c), full)


# ----------------------------------------------------------------------------- #
# rooted collectives
# ----------------------------------------------------------------------------- #
@pytest.mark.parametrize("root", [0, 2])
def test_rooted_collectives_against_their_unrooted_relatives(root):
    R, m = 4, 24
    x = inputs.rank_inputs(R, R * m, "bf16", seed=21)
    xi = inputs.rank_coded_i32(R, R * m)
    # reduce = the all-reduce result, at the root only
    red = oracle.reduce(x, root, "bf16")
    assert np.array_equal(red[root], oracle.allreduce(x, "bf16")[root])
    assert all(red[r] is None for r in range(R) if r != root)
    assert np.array_equal(oracle.reduce(xi, root, "i32")[root], oracle.allreduce(xi, "i32")[root])
    # gather = the all-gather result, at the root only
    g = oracle.gather(xi, root)
    assert np.array_equal(g[root], oracle.allgather(xi)[root]) and g[(root + 1) % R] is None
    # scatter = what all-to-all delivers from the root: partition r of the root's buffer
    sc = oracle.scatter(xi, root)
    a2a = oracle.alltoall(xi)
    for r in range(R):
        assert np.array_equal(sc[r], a2a[r][root * m:(root + 1) * m])
        assert sc[r][0] == root * R * m + r * m          # closed form on rank-coded ints
    # broadcast: every rank ends with the root's buffer; gather(scatter(x)) rebuilds it at the root
    bc = oracle.broadcast(xi, root)
    for r in range(R):
        assert np.array_equal(bc[r], xi[root])
    assert np.array_equal(oracle.gather(sc, root)[root], xi[root])


# ----------------------------------------------------------------------------- #
# MoE with per-rank deduplication
# ----------------------------------------------------------------------------- #
def test_moe_dedup_dispatch_and_combine():
    R, T, E, K, H = 4, 48, 16, 4, 8
    idx, _ = inputs.moe_routing(R, T, E, K, seed=12)
    epr = E // R
    x = [np.stack([np.full(2, p * 1000 + t, dtype=np.int32) for t in range(T)]) for p in range(R)]
    d = oracle.moe_dispatch_dedup(x, idx, E)
    plain = oracle.moe_dispatch(x, idx, E)
    for r in range(R):
        n = int(d["counts"][:, r].sum())
        meta = d["meta"][r][:n]
        # the (source, token) pairs that reach rank r: the distinct ones of the plain dispatch, in (p, t) order
        pm = plain["meta"][r][: int(plain["counts"][:, r].sum())]
        want = sorted({(int(a), int(b)) for a, b in pm[:, :2].tolist()})
        assert [tuple(v) for v in meta[:, :2].tolist()] == want
        assert np.array_equal(d["recv"][r][:n, 0], meta[:, 0] * 1000 + meta[:, 1])
        # the slot mask names exactly the slots whose expert lives on r
        for (p, t, mask, rr) in meta.tolist():
            assert rr == r and mask == sum(1 << j for j in range(K) if idx[p][t, j] // epr == r)
    # rows sent by p = number of distinct destination ranks over its tokens
    for p in range(R):
        distinct = sum(len(set((idx[p][t] // epr).tolist())) for t in range(T))
        assert int(d["counts"][p].sum()) == distinct
        assert distinct <= T * K
    # pos is the inverse map, -1 where the token does not go
    for p in range(R):
        for t in (0, T - 1):
            for r in range(R):
                row = d["pos"][p][t, r]
                assert (row >= 0) == (r in set((idx[p][t] // epr).tolist()))
                if row >= 0:
                    assert d["meta"][r][row][:2].tolist() == [p, t]
    # combine over identity rows: every destination returns the token, so out = (#ranks) * x
    xb = inputs.moe_tokens_bf16(R, T, H, seed=3)
    db = oracle.moe_dispatch_dedup(xb, idx, E)
    out = oracle.moe_combine_dedup(db["recv"], db["pos"], H)
    for p in range(R):
        nr = np.array([len(set((idx[p][t] // epr).tolist())) for t in range(T)], dtype=np.float64)
        assert np.array_equal(out[p], inputs.bf16_bits_to_f64(xb[p]) * nr[:, None])
    # one expert per rank and K = 1: deduplication changes nothing
    idx1 = [np.random.default_rng(p).integers(0, R, size=(T, 1)).astype(np.int32) for p in range(R)]
    a = oracle.moe_dispatch_dedup(x, idx1, R)
    b = oracle.moe_dispatch(x, idx1, R)
    for r in range(R):
        n = int(a["counts"][:, r].sum())
        assert np.array_equal(a["recv"][r][:n], b["recv"][r][:n]) and np.array_equal(a["counts"], b["counts"])


# ---- processing phase: scale, second operand, unconverted output ---------------------------------
def test_processed_sum_closed_forms():
    """Pins that a dropped term, a wrong sign or a scale applied to the wrong operand would break:
    residual = -sum gives exactly zero; equal inputs give R * x exactly (so the fp32 image of the
    result is R * x bit for bit); scale 1/R on equal inputs returns x; the residual is NOT scaled."""
    R, n = 8, 64
    ints = [gen.f32_to_bf16_bits(((np.arange(n) % 7) - 3 + r).astype(np.float32)) for r in range(R)]  # small integers: exact
    exact = sum(gen.bf16_bits_to_f64(a) for a in ints)
    res = [gen.f32_to_bf16_bits((-exact).astype(np.float32)) for _ in range(R)]
    assert np.array_equal(gen.bf16_bits_to_f64(res[0]), -exact)          # representable: |sum| <= 88
    out = oracle.allreduce_processed(ints, "bf16", 1.0, res)
    for r in range(R):
        assert np.all(out[r] == 0.0)
    x = gen.normal_bf16(n, 3, 0)
    same = [x.copy() for _ in range(R)]
    out = oracle.allreduce_processed(same, "bf16")
    assert np.array_equal(out[0], R * gen.bf16_bits_to_f64(x))
    assert np.array_equal(out[0].astype(np.float32).astype(np.float64), out[0])   # exact in fp32: R is a power of two
    out = oracle.allreduce_processed(same, "bf16", 1.0 / R)
    assert np.array_equal(out[5], gen.bf16_bits_to_f64(x))
    # scale applies to the sum only: with a zero sum the output is the second operand itself
    zero = [np.zeros(n, np.uint16) for _ in range(R)]
    aux = [gen.normal_bf16(n, 4, r) for r in range(R)]
    out = oracle.allreduce_processed(zero, "bf16", 0.125, aux)
    for r in range(R):
        assert np.array_equal(out[r], gen.bf16_bits_to_f64(aux[r]))
    # reduce-scatter form: rank r gets partition r, its own second operand, laid out like its output
    xs = [gen.normal_f32(R * 16, 9, r) for r in range(R)]
    aux = [gen.normal_f32(16, 10, r) for r in range(R)]
    out = oracle.reduce_scatter_processed(xs, "f32", 0.5, aux)
    stacked = np.stack([a.astype(np.float64) for a in xs]).sum(axis=0)
    for r in range(R):
        assert np.allclose(out[r], 0.5 * stacked[r * 16:(r + 1) * 16] + aux[r].astype(np.float64), rtol=0, atol=1e-12)
