"""Behaviour around the launch: a captured run replayed from a CUDA graph, the host-side table check in front of
the upload, and the sticky device status."""
import numpy as np
import pytest
import torch

import gpu_util as G
from paper_2609_34645_b200 import binding as B
from paper_2609_34645_b200 import inputs as I

pytestmark = pytest.mark.gpu


@pytest.mark.parametrize("variant,chained", [(1, False), (2, False), (3, False), (1, True), (2, True)])
def test_captured_run_replays_with_new_sources(variant, chained):
    """One run captured with cudaStreamBeginCapture and replayed three times, the sources refilled before each
    replay: every replay must move the new contents (the kernel leaves its control words zeroed for the next
    launch; nothing else is enqueued) and equal the oracle."""
    sh, a, b = I.SMALL, (2, 2), (4, 1)
    d = G.desc_of(sh)
    if chained:
        t = B.Transition.fuse([d.compile(B.Plan(*a), B.Plan(*b)), d.compile(B.Plan(*b), B.Plan(*a))], chained=True)
    else:
        t = d.compile(B.Plan(*a), B.Plan(*b))
    t.tune(variant=variant, tile_bytes=2048)
    t.prepare()                                                          # allocation stays out of the capture
    src = G.device_sources(d, B.Plan(*a), "bf16", 50)
    dst = G.Guarded([t.buffer_bytes(True, j) for j in range(t.num_buffers()[1])])
    stream = torch.cuda.Stream()
    sp, dp = [s.data_ptr() for s in src], dst.ptrs()
    with torch.cuda.stream(stream):
        t.run(sp, dp, stream.cuda_stream)                                # a plain run first
        stream.synchronize()
        g = torch.cuda.CUDAGraph()
        with torch.cuda.graph(g, stream=stream):
            t.run(sp, dp, stream.cuda_stream)
        for k in range(3):
            fresh = G.device_sources(d, B.Plan(*a), "bf16", 51 + k)
            for s, f in zip(src, fresh):
                s.copy_(f)
            for r in dst.raw:
                r.fill_(G.SENTINEL)
            g.replay()
            stream.synchronize()
            assert t.status() == B.DEV_OK
            want = G.oracle_expected(sh, a, b, "bf16", "bf16", False, [s.cpu().numpy() for s in src])
            for got, w in zip(dst.bufs[:4], want):
                assert np.array_equal(got.cpu().numpy(), w), k
            if chained:
                for got, s in zip(dst.bufs[4:], src):
                    assert torch.equal(got, s)
            assert dst.guards_intact()


def test_corrupted_table_is_refused_before_the_upload():
    d = G.desc_of(I.SMALL)
    t = d.compile(B.Plan(1, 1), B.Plan(4, 2))
    src = G.device_sources(d, B.Plan(1, 1), "bf16", 3)
    dst = G.Guarded([t.buffer_bytes(True, j) for j in range(8)])
    good = t.rects()[0]
    bad = t.rects()[0]
    bad.src_off = t.buffer_bytes(False, 0)                               # reads past the end of the source
    t.debug_set_rect(0, bad)
    assert t.prepare_raw() == B.ERR_TABLE
    assert t.run_raw([s.data_ptr() for s in src], dst.ptrs()) == B.ERR_TABLE
    torch.cuda.synchronize()
    assert t.launches() == 0
    for r in dst.raw:
        assert bool((r == G.SENTINEL).all())
    t.debug_set_rect(0, good)
    G.run_transition(t, src, dst.bufs)                                   # the repaired table runs
    with pytest.raises(B.NereusError) as e:
        t.debug_set_rect(0, bad)                                         # not once the table is on the device
    assert e.value.code == B.ERR_UNSUPPORTED


def test_run_with_declared_lengths():
    d = G.desc_of(I.SMALL)
    t = d.compile(B.Plan(2, 2), B.Plan(4, 1))
    src = G.device_sources(d, B.Plan(2, 2), "bf16", 4)
    dst = G.Guarded([t.buffer_bytes(True, j) for j in range(4)])
    sp, ss = [s.data_ptr() for s in src], [s.numel() for s in src]
    assert t.run_sized_raw(sp, ss, dst.ptrs(), [n - 16 for n in dst.sizes]) == B.ERR_TOO_SMALL
    torch.cuda.synchronize()
    assert t.launches() == 0 and all(bool((r == G.SENTINEL).all()) for r in dst.raw)
    assert t.run_sized_raw(sp, ss, dst.ptrs(), dst.sizes) == B.OK
    torch.cuda.synchronize()
    assert t.status() == B.DEV_OK
    want = G.oracle_expected(I.SMALL, (2, 2), (4, 1), "bf16", "bf16", False, [s.cpu().numpy() for s in src])
    for g, w in zip(dst.bufs, want):
        assert np.array_equal(g.cpu().numpy(), w)
    assert dst.guards_intact()


@pytest.mark.parametrize("variant,chained", [(1, False), (2, False), (3, False), (1, True), (2, True)])
def test_per_block_trace(variant, chained):
    """Tracing on: every tile is accounted to exactly one block, blocks start before they end, the result is
    still the oracle's; tracing off again: nothing to read."""
    sh, a, b = I.SMALL, (1, 1), (4, 2)
    d = G.desc_of(sh)
    t = d.compile(B.Plan(*a), B.Plan(*b))
    if chained:
        t = B.Transition.fuse([t, d.compile(B.Plan(*b), B.Plan(*a))], chained=True)
    t.tune(variant=variant, tile_bytes=2048)
    t.trace(True)
    src = G.device_sources(d, B.Plan(*a), "bf16", 21)
    dst = G.Guarded([t.buffer_bytes(True, j) for j in range(t.num_buffers()[1])])
    for _ in range(2):                                                   # the second run starts from an empty trace
        G.run_transition(t, src, dst.bufs)
    rec = t.trace_read()
    grid = t.launch_info()["grid"]
    assert 0 < len(rec) <= grid
    assert sum(r[3] for r in rec) == t.num_tiles()[0]
    busy = [r for r in rec if r[3]]
    assert all(r[2] >= r[1] > 0 for r in busy) and [r[0] for r in busy] == sorted({r[0] for r in busy})
    spread_us = (max(r[2] for r in busy) - min(r[1] for r in busy)) / 1e3
    assert 0 < spread_us < 1e5
    want = G.oracle_expected(sh, a, b, "bf16", "bf16", False, [s.cpu().numpy() for s in src])
    for g, w in zip(dst.bufs[:8], want):
        assert np.array_equal(g.cpu().numpy(), w)
    assert dst.guards_intact()
    t.trace(False)
    G.run_transition(t, src, dst.bufs)
    with pytest.raises(B.NereusError) as e:
        t.trace_read()
    assert e.value.code == B.ERR_ARG


def test_many_runs_back_to_back_need_no_reset():
    """200 launches of one handle without a synchronise in between: each finds the control words zeroed by the
    one before it."""
    d = G.desc_of(I.SMALL)
    for variant in (1, 2):
        t = d.compile(B.Plan(4, 2), B.Plan(1, 1))
        t.tune(variant=variant, tile_bytes=1024)
        src = G.device_sources(d, B.Plan(4, 2), "bf16", 9)
        dst = G.Guarded([t.buffer_bytes(True, 0)])
        stream = torch.cuda.current_stream()
        sp, dp = [s.data_ptr() for s in src], dst.ptrs()
        for k in range(200):
            if k == 199:
                dst.raw[0].fill_(G.SENTINEL)
            t.run(sp, dp, stream.cuda_stream)
        stream.synchronize()
        assert t.status() == B.DEV_OK and t.launches() == 200
        want = G.oracle_expected(I.SMALL, (4, 2), (1, 1), "bf16", "bf16", False, [s.cpu().numpy() for s in src])
        assert np.array_equal(dst.bufs[0].cpu().numpy(), want[0]) and dst.guards_intact()
