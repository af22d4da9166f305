"""Seeded random transitions on the GPU against the oracle: shapes, plans, layouts, dtypes, replica counts,
kernels and tile sizes drawn together, so that combinations no hand-written case lists are exercised."""
import random

import numpy as np
import pytest

import gpu_util as G
from oracle import oracle as O
from paper_2609_34645_b200 import binding as B
from paper_2609_34645_b200 import inputs as I

pytestmark = pytest.mark.gpu

SHAPES = [I.SMALL, I.MICRO, I.TINY, I.Shape(2, 128, 16, 2, 256, 256), I.Shape(3, 192, 6, 3, 384, 768),
          I.Shape(3, 192, 6, 6, 384, 768),              # 6 kv heads: TP 2 and 3 do not nest
          I.Shape(2, 64, 4, 4, 128, 1000),              # vocabulary that only tp 1, 2, 4 divide
          I.Shape(7, 64, 4, 4, 128, 256)]               # 7 layers: uneven pipeline cuts


def valid_plans(sh, padded=False):
    out = []
    for tp in (1, 2, 3, 4, 6, 8, 16):
        for pp in (1, 2, 3, 4, 8):
            kv_ok = sh.kv_heads % tp == 0 if tp <= sh.kv_heads else tp % sh.kv_heads == 0
            if kv_ok and sh.heads % tp == 0 and sh.ffn % tp == 0 and (padded or sh.vocab % tp == 0) \
                    and pp <= sh.layers:
                out.append((tp, pp))
    return out


def draw(rng):
    sh = rng.choice(SHAPES)
    pad_a, pad_b = (4 if rng.random() < 0.25 else 0), (4 if rng.random() < 0.25 else 0)   # padded vocabulary
    a, b = rng.choice(valid_plans(sh, pad_a)), rng.choice(valid_plans(sh, pad_b))
    sdt = rng.choice(["bf16", "bf16", "fp32"])
    ddt = "bf16" if sdt == "bf16" else rng.choice(["fp32", "bf16"])
    return dict(sh=sh, a=a, b=b, sdt=sdt, ddt=ddt, la=rng.randrange(4) | pad_a, lb=rng.randrange(4) | pad_b,
                vh=rng.random() < 0.25, k=rng.choice([1, 1, 1, 2, 3]), variant=rng.choice([1, 2, 3]),
                tile=rng.choice([512, 1024, 4096, 16384]))


@pytest.mark.parametrize("chunk", range(6))
def test_random_transitions(chunk):
    rng = random.Random(1000 + chunk)
    ran = 0
    for _ in range(14):
        c = draw(rng)
        sh = c["sh"]
        desc = G.desc_of(sh, c["sdt"], c["vh"])
        pa = B.Plan(c["a"][0], c["a"][1], 0, c["la"])
        pb = B.Plan(c["b"][0], c["b"][1], B.DTYPES[c["ddt"]], c["lb"])
        if c["variant"] == 2 and c["sdt"] != c["ddt"] and c["tile"] > 16384:
            continue
        try:
            t = desc.compile_replicated(pa, pb, c["k"])
        except B.NereusError as e:
            # pieces that are not multiples of 16 bytes are refused at compile time, never mis-copied
            assert e.code == B.ERR_INDIVISIBLE, c
            continue
        t.tune(tile_bytes=c["tile"], variant=c["variant"])
        oa = O.Plan(c["a"][0], c["a"][1], 0, c["la"])
        ob = O.Plan(c["b"][0], c["b"][1], G.ODT[c["ddt"]], c["lb"])
        src = G.device_sources_by_oracle(sh, oa, c["sdt"], 77 + ran, c["vh"])
        dst = G.Guarded([t.buffer_bytes(True, j) for j in range(t.num_buffers()[1])])
        G.run_transition(t, src, dst.bufs)
        want = O.reshard_replicated(G.omodel_of(sh, c["sdt"], c["vh"]), oa, ob, c["k"],
                                    [s.cpu().numpy() for s in src], fill=G.SENTINEL)
        for j, (g, w) in enumerate(zip(dst.bufs, want)):
            assert np.array_equal(g.cpu().numpy(), w), (c, j)
        assert dst.guards_intact(), c
        ran += 1
    assert ran >= 6


@pytest.mark.parametrize("chunk", range(3))
def test_random_chains(chunk):
    """Chains of two to four transitions fused into one table (one launch, dependency levels), through
    nereus_transition_run or through the allocation-free entry point: every intermediate layout and the last one
    against the oracle applied step by step."""
    import torch
    ran = 0
    for k in range(25):
        rng = random.Random(9000 + 100 * chunk + k)
        sh = rng.choice([I.SMALL, I.MICRO, I.TINY])
        chain = [rng.choice(valid_plans(sh)) for _ in range(rng.choice([2, 3, 3, 4]))]
        d = G.desc_of(sh)
        try:
            parts = [d.compile(B.Plan(*a), B.Plan(*b)) for a, b in zip(chain, chain[1:])]
        except B.NereusError as e:
            assert e.code == B.ERR_INDIVISIBLE, chain
            continue
        t = B.Transition.fuse(parts, chained=True) if len(parts) > 1 else parts[0]
        t.tune(variant=rng.choice([0, 1, 2]), tile_bytes=rng.choice([0, 512, 1024, 4096, 16384]))
        src = G.device_sources_by_oracle(sh, O.Plan(*chain[0]), "bf16", k)
        dst = G.Guarded([t.buffer_bytes(True, j) for j in range(t.num_buffers()[1])])
        stream = torch.cuda.current_stream()
        if rng.random() < 0.4 and len(t.rects()) <= B.STATIC_MAX_RECTS:
            t.run_static([s.data_ptr() for s in src], dst.ptrs(), stream.cuda_stream)
            stream.synchronize()
            assert B.static_status() == B.DEV_OK
        else:
            G.run_transition(t, src, dst.bufs)
        host, at, m = [s.cpu().numpy() for s in src], 0, G.omodel_of(sh)
        for a, b in zip(chain, chain[1:]):
            want = O.reshard(m, O.Plan(*a), O.Plan(*b), host, fill=G.SENTINEL)
            for g, w in zip(dst.bufs[at:at + len(want)], want):
                assert np.array_equal(g.cpu().numpy(), w), (chain, a, b)
            at, host = at + len(want), want
        assert dst.guards_intact(), chain
        ran += 1
    assert ran >= 10
