"""Pins for the seeded input generators (no method arithmetic is tested here)."""
import os

import numpy as np

from paper_2609_36954_b200 import inputs

GOLD = os.path.join(os.path.dirname(__file__), "golden")


def test_splitmix64_published_vector():
    # First outputs of the public-domain splitmix64 generator seeded with 0
    # (state advances by the golden gamma each call): a widely quoted test vector.
    s = np.uint64(0)
    got = []
    with np.errstate(over="ignore"):
        for _ in range(3):
            got.append(int(inputs.splitmix64(s)))
            s = s + inputs.GOLDEN
    assert got == [0xE220A8397B1DCDAF, 0x6E789E6AA1B965F4, 0x06C45D188009454F]


def test_uniform_grid_and_range():
    x = inputs.uniform_f32(1 << 16, 0, 3)
    assert x.dtype == np.float32 and x.min() >= -1.0 and x.max() < 1.0
    k = (x.astype(np.float64) + 1.0) * 2.0 ** 23
    assert np.all(k == np.round(k))  # exact 2^-23 grid
    assert abs(float(x.mean())) < 0.02
    # slices regenerate identically (counter based)
    assert np.array_equal(inputs.uniform_f32(100, 0, 3, start=500), x[500:600])


def test_normal_moments_and_streams_differ():
    z = inputs.normal_f64(1 << 18, 0, 0)
    assert abs(z.mean()) < 0.01 and abs(z.std() - 1.0) < 0.01
    b = inputs.normal_bf16(1 << 12, 0, 0)
    back = inputs.bf16_bits_to_f64(b)
    assert np.max(np.abs(back - z[: 1 << 12]) / np.maximum(np.abs(z[: 1 << 12]), 1e-30)) <= 2.0 ** -8
    assert not np.array_equal(b, inputs.normal_bf16(1 << 12, 0, 1))


def test_bf16_round_to_nearest_even():
    # 1 + 2^-8 is a tie between 1.0 and 1+2^-7 -> even mantissa (1.0);
    # 1 + 3*2^-8 is a tie between 1+2^-7 and 1+2^-6 -> even (1+2^-6)
    x = np.array([1.0 + 2.0 ** -8, 1.0 + 3 * 2.0 ** -8, 1.0 + 2.0 ** -8 + 2.0 ** -20], dtype=np.float32)
    got = inputs.bf16_bits_to_f32(inputs.f32_to_bf16_bits(x))
    assert got.tolist() == [1.0, 1.0 + 2.0 ** -6, 1.0 + 2.0 ** -7]


def test_zipf_split_matches_paper_statement():
    with open(os.path.join(GOLD, "zipf_split.txt")) as f:
        units = [int(v) for v in [l for l in f if not l.startswith("#")][0].split()]
    for logT in range(13, 31):
        T = 1 << logT
        n = inputs.zipf_split(T)
        u = max(128, T // 64)
        assert n.tolist() == [u * k for k in units]
        assert n.sum() == T and np.all(n % 128 == 0)
        assert n.max() == 1.125 * T / 8
    for T in (1024, 2048):
        assert inputs.zipf_split(T).tolist() == [T // 8] * 8
    for T in (4096,):
        n = inputs.zipf_split(T)
        assert n.sum() == T and np.all(n % 128 == 0)


def test_alltoallv_counts_send_and_receive_T():
    C = inputs.alltoallv_counts_bytes(1 << 20)
    assert np.all(C.sum(axis=1) == 1 << 20)
    assert np.all(C.sum(axis=0) == 1 << 20)


def test_moe_routing_shape_distinct_and_gates():
    R, T, E, K = 4, 256, 64, 8
    idx, gates = inputs.moe_routing(R, T, E, K)
    for r in range(R):
        assert idx[r].shape == (T, K) and idx[r].dtype == np.int32
        assert idx[r].min() >= 0 and idx[r].max() < E
        assert all(len(set(row)) == K for row in idx[r].tolist())
        assert gates[r].dtype == np.float32
        assert np.allclose(gates[r].sum(axis=1), 1.0, atol=1e-6)
        assert np.all(np.diff(gates[r], axis=1) <= 0)  # slot order = descending logit
    # skew: the hottest expert draws far more rows than the mean
    h = np.bincount(np.concatenate([i.ravel() for i in idx]), minlength=E)
    assert h.max() > 3 * h.mean()
    idx2, _ = inputs.moe_routing(R, T, E, K, identity_perm=True)
    h2 = np.bincount(np.concatenate([i.ravel() for i in idx2]), minlength=E)
    assert h2[:8].sum() > h2[-8:].sum() * 4  # identity map: low ids are the hot ones
