"""Seeded synthetic inputs for the collectives executor (numpy only).

This module holds the counter-based generators that feed BOTH the CUDA path and
the test oracle.  It contains none of the method's arithmetic (no reduction, no
permutation of rank buffers, no dispatch/combine): it only draws numbers, and for
the MoE workload it draws a routing table (expert ids + gates), which the method
takes as an input.

Generator: ``key = splitmix64(seed ^ (GOLDEN * (stream + 1)))`` and
``h(c) = splitmix64(key + c)``; every draw is a pure function of
``(seed, stream, counter)``, so any slice of any buffer can be regenerated.

Workload shapes follow the paper's evaluation: BF16 reductions, 8 ranks,
power-of-two message sweep (Sec. 5, "Microbenchmark methodology"), expert-parallel
dispatch/combine (Table 2), and the Zipf(s=0.125) variable-length split
(Appendix C, Eq. "zipf-split").
"""
from __future__ import annotations

import numpy as np

GOLDEN = np.uint64(0x9E3779B97F4A7C15)
_M1 = np.uint64(0xBF58476D1CE4E5B9)
_M2 = np.uint64(0x94D049BB133111EB)
_BLOCK = 1 << 22  # elements generated per numpy pass (bounds temporaries)


def splitmix64(x):
    """One splitmix64 output step on uint64 scalars/arrays (wrapping arithmetic)."""
    with np.errstate(over="ignore"):
        z = np.asarray(x, dtype=np.uint64) + GOLDEN
        z = (z ^ (z >> np.uint64(30))) * _M1
        z = (z ^ (z >> np.uint64(27))) * _M2
        return z ^ (z >> np.uint64(31))


def stream_key(seed: int, stream: int) -> np.uint64:
    with np.errstate(over="ignore"):
        k = np.uint64(seed) ^ (GOLDEN * np.uint64(stream + 1))
    return splitmix64(k)


def hash_counter(seed: int, stream: int, counters) -> np.ndarray:
    """h(c) for an array of counters."""
    key = stream_key(seed, stream)
    with np.errstate(over="ignore"):
        return splitmix64(key + np.asarray(counters, dtype=np.uint64))


# --------------------------------------------------------------------------- #
# dtype helpers (bf16 is carried as uint16 bit patterns)
# --------------------------------------------------------------------------- #
def f32_to_bf16_bits(x: np.ndarray) -> np.ndarray:
    """Round-to-nearest-even fp32 -> bf16 bit pattern (finite inputs)."""
    u = np.ascontiguousarray(x, dtype=np.float32).view(np.uint32)
    r = u + np.uint32(0x7FFF) + ((u >> np.uint32(16)) & np.uint32(1))
    return (r >> np.uint32(16)).astype(np.uint16)


def bf16_bits_to_f32(b: np.ndarray) -> np.ndarray:
    return (np.ascontiguousarray(b, dtype=np.uint16).astype(np.uint32) << np.uint32(16)).view(np.float32)


def bf16_bits_to_f64(b: np.ndarray) -> np.ndarray:
    return bf16_bits_to_f32(b).astype(np.float64)


# --------------------------------------------------------------------------- #
# value streams
# --------------------------------------------------------------------------- #
def uniform_f32(n: int, seed: int, stream: int, start: int = 0) -> np.ndarray:
    """fp32 uniform on the 2^-23 grid in [-1, 1): (h(i) >> 40) * 2^-23 - 1."""
    out = np.empty(n, dtype=np.float32)
    for b in range(0, n, _BLOCK):
        m = min(_BLOCK, n - b)
        c = np.arange(start + b, start + b + m, dtype=np.uint64)
        h = hash_counter(seed, stream, c)
        out[b:b + m] = ((h >> np.uint64(40)).astype(np.float64) * 2.0 ** -23 - 1.0).astype(np.float32)
    return out


def normal_f64(n: int, seed: int, stream: int, start: int = 0) -> np.ndarray:
    """Box-Muller N(0,1) in fp64 from counters 2i and 2i+1."""
    out = np.empty(n, dtype=np.float64)
    for b in range(0, n, _BLOCK):
        m = min(_BLOCK, n - b)
        i = np.arange(start + b, start + b + m, dtype=np.uint64)
        h1 = hash_counter(seed, stream, i * np.uint64(2))
        h2 = hash_counter(seed, stream, i * np.uint64(2) + np.uint64(1))
        u1 = ((h1 >> np.uint64(40)).astype(np.float64) + 1.0) * 2.0 ** -24
        u2 = (h2 >> np.uint64(40)).astype(np.float64) * 2.0 ** -24
        out[b:b + m] = np.sqrt(-2.0 * np.log(u1)) * np.cos(2.0 * np.pi * u2)
    return out


def normal_bf16(n: int, seed: int, stream: int, start: int = 0) -> np.ndarray:
    """N(0,1) rounded RNE to bf16; returned as uint16 bit patterns."""
    out = np.empty(n, dtype=np.uint16)
    for b in range(0, n, _BLOCK):
        m = min(_BLOCK, n - b)
        z = normal_f64(m, seed, stream, start + b)
        out[b:b + m] = f32_to_bf16_bits(z.astype(np.float32))
    return out


def normal_f32(n: int, seed: int, stream: int, start: int = 0) -> np.ndarray:
    return normal_f64(n, seed, stream, start).astype(np.float32)


def rank_coded_i32(R: int, n: int) -> list:
    """int32 twin of an allreduce input: x[r][i] = r*n + i."""
    base = np.arange(n, dtype=np.int64)
    return [(base + r * n).astype(np.int32) for r in range(R)]


def rank_coded_bytes(R: int, nbytes: int) -> list:
    """Byte buffers whose content identifies (rank, position): a 1:1 hash byte."""
    out = []
    for r in range(R):
        i = np.arange(nbytes, dtype=np.uint64)
        out.append((hash_counter(0x5EED, r, i) & np.uint64(0xFF)).astype(np.uint8))
    return out


def rank_inputs(R: int, n: int, dtype: str, seed: int = 0, stream_base: int = 0) -> list:
    """Per-rank input buffers of n elements: 'bf16' -> uint16 bits of N(0,1),
    'f32' -> uniform grid in [-1,1), 'f32n' -> N(0,1) fp32, 'i32' -> rank coded."""
    if dtype == "bf16":
        return [normal_bf16(n, seed, stream_base + r) for r in range(R)]
    if dtype == "f32":
        return [uniform_f32(n, seed, stream_base + r) for r in range(R)]
    if dtype == "f32n":
        return [normal_f32(n, seed, stream_base + r) for r in range(R)]
    if dtype == "i32":
        return rank_coded_i32(R, n)
    raise ValueError(dtype)


# --------------------------------------------------------------------------- #
# variable-length split (Appendix C, Eq. "zipf-split")
# --------------------------------------------------------------------------- #
def zipf_split(T: int, W: int = 8, s: float = 0.125) -> np.ndarray:
    """Bytes n_r assigned to rank r out of T total: unit u = max(128, T/(8W)),
    x_r = (T/u) (r+1)^-s / sum_k (k+1)^-s, n_r = u (floor(x_r) + delta_r) with the
    leftover units handed out by descending fractional part, ties to lower rank.
    Totals too small to give every rank one unit are split uniformly."""
    u = max(128, T // (8 * W))
    units = T // u
    if units < 8 * W:  # 1-2 KiB totals at W=8: the paper rounds these to uniform
        assert T % W == 0
        return np.full(W, T // W, dtype=np.int64)
    w = np.array([(r + 1.0) ** -s for r in range(W)], dtype=np.float64)
    x = units * w / w.sum()
    fl = np.floor(x).astype(np.int64)
    left = int(units - fl.sum())
    frac = x - fl
    order = sorted(range(W), key=lambda r: (-frac[r], r))
    for r in order[:left]:
        fl[r] += 1
    return fl * u


def alltoallv_counts_bytes(T: int, W: int = 8) -> np.ndarray:
    """C[p][r] bytes sent from p to r: the Zipf split rotated right by (p+1) mod W
    at rank p, so that every rank sends and receives T bytes."""
    n = zipf_split(T, W)
    C = np.zeros((W, W), dtype=np.int64)
    for p in range(W):
        C[p] = np.roll(n, (p + 1) % W)
    return C


# --------------------------------------------------------------------------- #
# MoE routing (expert-parallel dispatch/combine workload)
# --------------------------------------------------------------------------- #
def expert_permutation(E: int, seed: int = 1) -> np.ndarray:
    """pi[e] = popularity rank (0 = hottest) of expert id e: seeded shuffle."""
    keys = hash_counter(seed, 0x70, np.arange(E, dtype=np.uint64))
    order = np.argsort(keys, kind="stable")  # order[k] = expert id with popularity rank k
    pi = np.empty(E, dtype=np.int64)
    pi[order] = np.arange(E)
    return pi


def moe_routing(R: int, T: int, E: int, K: int, zipf_s: float = 1.2, seed: int = 0,
                identity_perm: bool = False, perm_seed: int = 1):
    """Top-K routing with Zipf(s) expert popularity via Gumbel top-k.

    Returns (idx, gates): idx[r] int32 [T,K] distinct expert ids per token, slot
    order = descending perturbed logit (ties to the lower expert id); gates[r]
    fp32 [T,K] = softmax (max-subtracted, fp32) over the K selected logits.
    """
    pop = np.arange(1, E + 1, dtype=np.float64) ** -zipf_s
    pop /= pop.sum()
    pi = np.arange(E) if identity_perm else expert_permutation(E, perm_seed)
    logp = np.log(pop)[pi]
    idx_all, gate_all = [], []
    for r in range(R):
        c = (np.uint64(r * T) + np.arange(T, dtype=np.uint64))[:, None] * np.uint64(E) \
            + np.arange(E, dtype=np.uint64)[None, :]
        h = hash_counter(seed, 0x40E, c)
        u = ((h >> np.uint64(40)).astype(np.float64) + 0.5) * 2.0 ** -24
        logits = logp[None, :] - np.log(-np.log(u))
        # stable sort on -logits: ties resolve to the lower expert id
        order = np.argsort(-logits, axis=1, kind="stable")[:, :K]
        sel = np.take_along_axis(logits, order, axis=1).astype(np.float32)
        ex = np.exp(sel - sel.max(axis=1, keepdims=True), dtype=np.float32)
        gates = (ex / ex.sum(axis=1, keepdims=True, dtype=np.float32)).astype(np.float32)
        idx_all.append(np.ascontiguousarray(order.astype(np.int32)))
        gate_all.append(np.ascontiguousarray(gates))
    return idx_all, gate_all


def moe_tokens_bf16(R: int, T: int, H: int, seed: int = 2) -> list:
    return [normal_bf16(T * H, seed, r).reshape(T, H) for r in range(R)]
