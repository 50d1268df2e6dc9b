"""Test tool: replays a dumped schedule on the CPU with numpy.

It is neither the oracle nor the product: it executes the op list produced by the host
orchestrator (pl_schedule_dump) queue by queue in a *random* interleaving that honours only
the wait/signal edges, over poison-filled output and scratch buffers.  A missing dependency
edge therefore shows up as a wrong result (or as a deadlock) without any GPU.
"""
from __future__ import annotations

import random

import numpy as np

from paper_2609_36954_b200 import binding as B
from paper_2609_36954_b200 import inputs as gen

_ES = {B.PL_BF16: 2, B.PL_F32: 4, B.PL_I32: 4, B.PL_U8: 1, B.PL_F32X2: 8}


def _load(buf, off, count, dtype):
    raw = buf[off:off + count * _ES[dtype]]
    if dtype == B.PL_BF16:
        return gen.bf16_bits_to_f32(raw.view(np.uint16))
    if dtype == B.PL_F32:
        return raw.view(np.float32).copy()
    if dtype == B.PL_I32:
        return raw.view(np.uint32).copy()
    if dtype == B.PL_F32X2:  # blocks of 4 sums then 4 corrections; value = sum + correction
        blk = raw.view(np.float32).reshape(-1, 2, 4).astype(np.float64)
        return (blk[:, 0, :] + blk[:, 1, :]).reshape(-1)
    return raw.copy()


def _store(buf, off, vals, dtype):
    if dtype == B.PL_BF16:
        raw = gen.f32_to_bf16_bits(vals.astype(np.float32)).view(np.uint8)
    elif dtype == B.PL_F32:
        raw = vals.astype(np.float32).view(np.uint8)
    elif dtype == B.PL_I32:
        raw = vals.astype(np.uint32).view(np.uint8)
    elif dtype == B.PL_F32X2:
        v = vals.astype(np.float64).reshape(-1, 4)
        hi = v.astype(np.float32)
        lo = (v - hi.astype(np.float64)).astype(np.float32)
        raw = np.stack([hi, lo], axis=1).reshape(-1).view(np.uint8)
    else:
        raw = vals
    buf[off:off + raw.size] = raw


def run(ops, info, R, ins, seed=0, max_steps=None, aux=None, scale=1.0, elem_dtype=None):
    """ins[r]: numpy arrays (any dtype).  Returns list of uint8 output buffers.  aux / scale /
    elem_dtype: second operand per rank (element-typed, laid out like the output), output scale and
    element type of a schedule with a processing phase (applied by ops flagged final)."""
    rng = random.Random(seed)
    bufs = {B.PL_BUF_IN: [np.ascontiguousarray(a).view(np.uint8).reshape(-1) for a in ins],
            B.PL_BUF_OUT: [np.full(int(info.out_bytes[r]), 0xFF, np.uint8) for r in range(R)],
            B.PL_BUF_SCRATCH: [np.full(int(info.scratch_bytes) + 16, 0xFF, np.uint8) for _ in range(R)]}
    for r in range(R):
        assert bufs[B.PL_BUF_IN][r].size >= int(info.in_bytes[r])
    nq = int(info.n_queues)
    queues = [[] for _ in range(nq)]
    for op in sorted(ops, key=lambda o: o.topo):
        queues[op.queue].append(op)
    heads = [0] * nq
    flags = [0] * int(info.n_flags)
    remaining = len(ops)
    while remaining:
        runnable = []
        for q in range(nq):
            if heads[q] < len(queues[q]):
                op = queues[q][heads[q]]
                if all(flags[op.wait_flag[k]] >= op.wait_need[k] for k in range(op.n_wait)):
                    runnable.append(q)
        if not runnable:
            raise AssertionError("schedule deadlocks: no queue head is runnable")
        q = rng.choice(runnable)
        op = queues[q][heads[q]]
        heads[q] += 1
        remaining -= 1
        n = int(op.count)
        if op.kind == B.PL_OP_COPY:
            data = _load(bufs[op.src[0].buf][op.src[0].rank], int(op.src[0].offset), n, B.PL_U8)
            result, rdt = data, B.PL_U8
        else:
            first = op.src[0]
            kinds = {op.src[k].dtype for k in range(op.n_src)} | {op.dst.dtype}
            if first.dtype == B.PL_I32:
                acc = np.zeros(n, np.uint32)
            elif B.PL_F32X2 in kinds or B.PL_F32 in kinds:
                acc = np.zeros(n, np.float64)  # stands in for the compensated fp32 (sum, correction) pair
            else:
                acc = np.zeros(n, np.float32)
            for k in range(op.n_src):
                s = op.src[k]
                acc = acc + _load(bufs[s.buf][s.rank], int(s.offset), n, s.dtype)
            result, rdt = acc, op.dst.dtype
        targets = range(R) if (op.dst_bcast & 1) else [op.dst.rank]
        final = bool(op.dst_bcast & 2)
        for r in targets:
            val = result
            if final:
                val = np.float64(scale) * result.astype(np.float64)
                if aux is not None:  # the second operand is element-typed and indexed like the (unconverted) output
                    e_off = int(op.dst.offset) // _ES[rdt] * _ES[elem_dtype]
                    val = val + _load(np.ascontiguousarray(aux[r]).view(np.uint8).reshape(-1), e_off, n, elem_dtype).astype(np.float64)
            _store(bufs[op.dst.buf][r], int(op.dst.offset), val, rdt)
        for f in (op.signal_flag, op.signal_flag2):
            if f >= 0:
                flags[f] += 1
    return bufs[B.PL_BUF_OUT]


def run_two_overlapped(ops, info, R, ins_a, ins_b, seed=0):
    """Two back-to-back executes of a schedule built with two staging buffers (PL_OPT_STAGE_AHEAD).
    Execute B's early stage ops (flag value 4 in dst_bcast; only the leading ones of a queue) may
    interleave freely with execute A's ops; everything else of B starts when A has finished.  Each
    execute has its own staging memory and flag set (launch parity); they share the output buffers.
    Returns (outputs after A, outputs after B)."""
    rng = random.Random(seed)
    nq = int(info.n_queues)
    queues = [[] for _ in range(nq)]
    for op in sorted(ops, key=lambda o: o.topo):
        queues[op.queue].append(op)
    outs = [np.full(int(info.out_bytes[r]), 0xFF, np.uint8) for r in range(R)]

    class Exe:
        def __init__(self, ins):
            self.bufs = {B.PL_BUF_IN: [np.ascontiguousarray(a).view(np.uint8).reshape(-1) for a in ins], B.PL_BUF_OUT: outs,
                         B.PL_BUF_SCRATCH: [np.full(int(info.scratch_bytes) + 16, 0xFF, np.uint8) for _ in range(R)]}
            self.heads = [0] * nq
            self.flags = [0] * int(info.n_flags)
            self.left = len(ops)

        def runnable(self, early_only):
            out = []
            for q in range(nq):
                if self.heads[q] < len(queues[q]):
                    op = queues[q][self.heads[q]]
                    if early_only and not (op.dst_bcast & 4):
                        continue
                    if all(self.flags[op.wait_flag[k]] >= op.wait_need[k] for k in range(op.n_wait)):
                        out.append(q)
            return out

        def step(self, q):
            op = queues[q][self.heads[q]]
            self.heads[q] += 1
            self.left -= 1
            n = int(op.count)
            if op.kind == B.PL_OP_COPY:
                result, rdt = _load(self.bufs[op.src[0].buf][op.src[0].rank], int(op.src[0].offset), n, B.PL_U8), B.PL_U8
            else:
                first = op.src[0]
                acc = np.zeros(n, np.uint32 if first.dtype == B.PL_I32 else np.float32)
                for k in range(op.n_src):
                    sk = op.src[k]
                    acc = acc + _load(self.bufs[sk.buf][sk.rank], int(sk.offset), n, sk.dtype)
                result, rdt = acc, op.dst.dtype
            for r in (range(R) if (op.dst_bcast & 1) else [op.dst.rank]):
                _store(self.bufs[op.dst.buf][r], int(op.dst.offset), result, rdt)
            for f in (op.signal_flag, op.signal_flag2):
                if f >= 0:
                    self.flags[f] += 1

    a, b = Exe(ins_a), Exe(ins_b)
    early_steps = 0
    while a.left:
        ra, rb = a.runnable(False), b.runnable(True)
        assert ra, "execute A deadlocks"
        if rb and rng.random() < 0.5:
            b.step(rng.choice(rb))
            early_steps += 1
        else:
            a.step(rng.choice(ra))
    after_a = [o.copy() for o in outs]
    for o in outs:
        o[:] = 0xFF
    while b.left:
        rb = b.runnable(False)
        assert rb, "execute B deadlocks"
        b.step(rng.choice(rb))
    return after_a, [o.copy() for o in outs], early_steps
