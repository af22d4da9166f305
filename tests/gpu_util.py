"""Helpers of the GPU parity tests: seeded device inputs laid out through the library's own layout query,
destination buffers with sentinel fill and guard zones, and the comparison with the CPU oracle."""
from __future__ import annotations

import os
from concurrent.futures import ThreadPoolExecutor

import numpy as np
import torch

from oracle import oracle as O
from paper_2609_34645_b200 import binding as B
from paper_2609_34645_b200 import inputs as I

GUARD = 4096
SENTINEL = 0xA5
ODT = {"bf16": O.BF16, "fp32": O.FP32}


def desc_of(sh, dtype="bf16", value_head=False):
    return B.ModelDesc(sh.layers, sh.hidden, sh.heads, sh.kv_heads, sh.ffn, sh.vocab, B.DTYPES[dtype], value_head)


def omodel_of(sh, dtype="bf16", value_head=False):
    return O.Model(sh.layers, sh.hidden, sh.heads, sh.kv_heads, sh.ffn, sh.vocab, ODT[dtype], value_head)


def replica_groups(desc, plan):
    """Byte ranges of replicated tensors, grouped per tensor and pipeline stage, from the library's query."""
    n = desc.num_shards(plan)
    groups = []
    for tid in range(desc.num_tensors()):
        grp = []
        for s in range(n):
            off, rows, cols, rep = desc.tensor_slice(plan, s, tid)
            if rep and rows:
                grp.append((s, off, rows * cols))        # (shard, byte offset, elements)
        if len(grp) > 1:
            groups.append(grp)
    return groups


def device_sources(desc, plan, dtype, seed, device="cuda"):
    """Seeded N(0, 0.02) source shards on the device with replicated tensors tied."""
    sizes = desc.shard_sizes(plan)
    bufs = I.make_shards(sizes, dtype, seed, device)
    es = I.element_size(dtype)
    groups = [[(s, off, n * es) for s, off, n in g] for g in replica_groups(desc, plan)]
    I.tie_replicas(bufs, groups)
    return bufs


def device_sources_by_oracle(sh, plan, dtype, seed, value_head=False, device="cuda"):
    """Same, with the copies found through the oracle's layout: every region that several shards hold (norms,
    value head, kv heads when tp > kv_heads) is tied.  plan = oracle Plan."""
    m = omodel_of(sh, dtype, value_head)
    n = O.num_shards(m, plan)
    bufs = I.make_shards([O.shard_bytes(m, plan, s) for s in range(n)], dtype, seed, device)
    groups = []
    for t in range(O.num_logical(m)):
        same = {}
        for s in range(n):
            p = O.locate(m, plan, s, t)
            if p.held:
                same.setdefault((p.r0, p.c0, p.nr, p.nc), []).append((s, p.offset, p.nr * p.nc * O.es(m, plan)))
        groups += [g for g in same.values() if len(g) > 1]
    I.tie_replicas(bufs, groups)
    return bufs


class Guarded:
    """Destination buffers with a guard zone on both sides, all pre-filled with a sentinel byte."""

    def __init__(self, sizes, device="cuda"):
        self.sizes = [int(s) for s in sizes]
        self.raw = [torch.full((s + 2 * GUARD,), SENTINEL, dtype=torch.uint8, device=device) for s in self.sizes]
        self.bufs = [r[GUARD:GUARD + s] for r, s in zip(self.raw, self.sizes)]

    def ptrs(self):
        return [b.data_ptr() for b in self.bufs]

    def guards_intact(self):
        for r, s in zip(self.raw, self.sizes):
            if not bool((r[:GUARD] == SENTINEL).all()) or not bool((r[GUARD + s:] == SENTINEL).all()):
                return False
        return True


def run_transition(t, src_bufs, dst_bufs, stream=None):
    stream = stream or torch.cuda.current_stream()
    t.run([b.data_ptr() for b in src_bufs], [b.data_ptr() for b in dst_bufs], stream.cuda_stream)
    stream.synchronize()
    assert t.status() == B.DEV_OK


def oracle_expected(sh, a, b, sdt, ddt, vh, src_host):
    m = omodel_of(sh, sdt, vh)
    return O.reshard(m, O.Plan(*a), O.Plan(b[0], b[1], ODT[ddt]), src_host, fill=SENTINEL)


def check_against_oracle(sh, a, b, sdt="bf16", ddt="bf16", vh=False, seed=0, tune=None):
    """Full element-by-element parity of one transition, padding and guard zones included."""
    desc = desc_of(sh, sdt, vh)
    pa, pb = B.Plan(*a), B.Plan(b[0], b[1], B.DTYPES[ddt])
    t = desc.compile(pa, pb)
    if tune:
        t.tune(**tune)
    src = device_sources(desc, pa, sdt, seed)
    dst = Guarded([t.buffer_bytes(True, j) for j in range(t.num_buffers()[1])])
    before = t.launches()
    run_transition(t, src, dst.bufs)
    assert t.launches() == before + 1
    want = oracle_expected(sh, a, b, sdt, ddt, vh, [s.cpu().numpy() for s in src])
    for j, (g, w) in enumerate(zip(dst.bufs, want)):
        g = g.cpu().numpy()
        if not np.array_equal(g, w):
            bad = np.flatnonzero(g != w)
            raise AssertionError(f"{a}->{b} shard {j}: {bad.size} bytes differ, first at {bad[0]}")
    assert dst.guards_intact()
    return t


# ---------------------------------------------------------------- every logical tensor, at any size

def host_workers() -> int:
    """Threads the full-size comparisons may use: the cores this process may run on, at most 32."""
    try:
        n = len(os.sched_getaffinity(0))
    except AttributeError:
        n = os.cpu_count() or 1
    return max(1, min(32, n))


def _span_bytes(m, plan, tid, part, es):
    """Bytes from the first element of a shard's part of logical tensor tid to the end of its last row (the
    rows of a part are interleaved with other tensors' rows under the grouped and interleaved layouts)."""
    if not part.held:
        return 0
    return (O.part_row(m, plan, tid, part.nr - 1) + 1) * part.nc * es


def _compare_one_tensor(m, pa, pb, tid, src, dst_units, ses, des):
    """One logical tensor through the oracle, from device slices of the sources, against the device result of
    every destination unit.  The oracle (single-threaded, as it stands) writes the tensor's rows over a host copy
    of what the device holds in the span of each part: equal afterwards means every element was right."""
    ns, nd = O.num_shards(m, pa), O.num_shards(m, pb)
    sparts = []
    for s in range(ns):
        p = O.locate(m, pa, s, tid)
        n = _span_bytes(m, pa, tid, p, ses)
        sparts.append(src[s][p.offset:p.offset + n].cpu().numpy() if p.held else None)
    where = [O.locate(m, pb, d, tid) for d in range(nd)]
    spans = [_span_bytes(m, pb, tid, p, des) for p in where]
    first = dst_units[0]
    got = [first[d][p.offset:p.offset + n].cpu().numpy() if p.held else None for d, (p, n) in enumerate(zip(where, spans))]
    want = [None if g is None else g.copy() for g in got]
    O.reshard_tensor_parts(m, pa, pb, tid, sparts, want)
    compared = 0
    for d, (g, w) in enumerate(zip(got, want)):
        if g is None:
            continue
        if not np.array_equal(g, w):
            bad = np.flatnonzero(g != w)
            return f"logical tensor {tid}, destination shard {d}: {bad.size} bytes differ, first at {int(bad[0])}"
        compared += g.size
    # further units (replicas) hold what the first one holds, byte for byte
    for k, dst in enumerate(dst_units[1:], 1):
        for d, (p, n) in enumerate(zip(where, spans)):
            if p.held and not torch.equal(dst[d][p.offset:p.offset + n], first[d][p.offset:p.offset + n]):
                return f"logical tensor {tid}, unit {k}, destination shard {d} differs from unit 0"
            compared += n if p.held else 0
    return compared


def compare_every_tensor(jobs, workers=None):
    """jobs: iterable of (model, src plan, dst plan, source buffers, [destination units]) with device buffers
    (torch uint8) and oracle-side models and plans.  EVERY logical tensor of every job goes through the oracle
    and is compared element by element with the device result; disjoint tensors run on a pool of host threads
    (each oracle call is the single-threaded C routine; ctypes and the copies release the interpreter lock).
    Returns the destination bytes compared; raises AssertionError on the first difference."""
    tasks = []
    for m, pa, pb, src, dst_units in jobs:
        ses, des = O.es(m, pa), O.es(m, pb)
        for tid in range(O.num_logical(m)):
            rows, cols = O.logical_shape(m, tid)
            tasks.append((rows * cols, m, pa, pb, tid, src, dst_units, ses, des))
    tasks.sort(key=lambda x: -x[0])                         # the embeddings first: they take the longest
    total = 0
    with ThreadPoolExecutor(max_workers=workers or host_workers()) as pool:
        for res in pool.map(lambda a: _compare_one_tensor(*a[1:]), tasks):
            assert not isinstance(res, str), res
            total += res
    return total
