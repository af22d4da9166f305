"""The allocation-free entry point, nereus_transition_run_static, against nereus_transition_run and the oracle.

It serves callers that cannot allocate device memory when a transition is due (their own pool owns the
GPU), so its task table lives in a fixed device array that all calls share.  The tests call it through the C
ABI: twice in a row with two different transitions, so that the second call must overwrite what the first one
left in the array, asking for bit-identical destinations (the tolerance of every reshard test: none) against
the allocating entry point and against the CPU oracle; through the shared-memory ring and through a chained
two-level table; with the device's free memory read before and after; and with a dependency wait that is
made to give up, whose status only nereus_static_status can report.
Collected last on purpose: a failure here stops nothing else.
"""
import numpy as np
import pytest
import torch

import gpu_util as G
from paper_2609_34645_b200 import binding as B
from paper_2609_34645_b200 import inputs as I

pytestmark = pytest.mark.gpu


def _pair(sh, a, b, sdt, ddt, seed):
    desc = G.desc_of(sh, sdt)
    pa, pb = B.Plan(*a), B.Plan(b[0], b[1], B.DTYPES[ddt])
    t = desc.compile(pa, pb)
    src = G.device_sources(desc, pa, sdt, seed)
    sizes = [t.buffer_bytes(True, j) for j in range(t.num_buffers()[1])]
    return desc, t, src, sizes


CASES = [(I.SMALL, (1, 1), (4, 2), "bf16", "bf16", 31),        # Split, many pitched tasks
         (I.SMALL, (2, 2), (4, 1), "fp32", "bf16", 32)]        # cast, a different and shorter table


def _assert_equals_oracle(case, src, out):
    sh, a, b, sdt, ddt, _ = case
    want = G.oracle_expected(sh, a, b, sdt, ddt, False, [s.cpu().numpy() for s in src])
    for g, w in zip(out.bufs, want):
        assert np.array_equal(g.cpu().numpy(), w)
    assert out.guards_intact()


def test_run_static_matches_run_twice_in_a_row():
    assert torch.cuda.is_available()
    stream = torch.cuda.current_stream()
    cases = [_pair(*c) for c in CASES]
    ref, got = [], []
    for desc, t, src, sizes in cases:
        want = G.Guarded(sizes)
        G.run_transition(t, src, want.bufs)                              # existing entry point
        ref.append(want)
    for desc, t, src, sizes in cases:                                    # two static calls, back to back
        out = G.Guarded(sizes)
        t.run_static([s.data_ptr() for s in src], out.ptrs(), stream.cuda_stream)
        got.append(out)
    stream.synchronize()
    assert B.static_status() == B.DEV_OK
    for case, (desc, t, src, sizes), want, out in zip(CASES, cases, ref, got):
        for w, g in zip(want.raw, out.raw):                              # payload, padding and guard zones
            assert torch.equal(w, g)
        _assert_equals_oracle(case, src, out)
    # once more in the opposite order: the first table must be restored over the second
    for (desc, t, src, sizes), want in reversed(list(zip(cases, ref))):
        out = G.Guarded(sizes)
        t.run_static([s.data_ptr() for s in src], out.ptrs(), stream.cuda_stream)
        stream.synchronize()
        for w, g in zip(want.raw, out.raw):
            assert torch.equal(w, g)


@pytest.mark.parametrize("case", CASES)
def test_run_static_through_the_ring(case):
    """The shared-memory ring (forced: tables this small default to the vector kernel) from the fixed array."""
    desc, t, src, sizes = _pair(*case)
    t.tune(variant=2)
    assert t.launch_info()["kernel"] == "nereus_walk_ring"
    stream = torch.cuda.current_stream()
    for _ in range(2):
        out = G.Guarded(sizes)
        t.run_static([s.data_ptr() for s in src], out.ptrs(), stream.cuda_stream)
        stream.synchronize()
        assert B.static_status() == B.DEV_OK
        _assert_equals_oracle(case, src, out)


@pytest.mark.parametrize("variant", [1, 2])
def test_run_static_chained_round_trip_and_its_status(variant, monkeypatch):
    """A two-level table (there and back) from the fixed array: level 1 waits for level 0 through the control
    words that live in that array too.  Then the wait is made to give up (a gate nothing opens): the call still
    returns, and nereus_static_status reports the timeout once, nereus_transition_status never sees it."""
    sh, a, b = I.SMALL, (2, 2), (4, 1)
    d = G.desc_of(sh)
    t = B.Transition.fuse([d.compile(B.Plan(*a), B.Plan(*b)), d.compile(B.Plan(*b), B.Plan(*a))], chained=True)
    t.tune(variant=variant)
    src = G.device_sources(d, B.Plan(*a), "bf16", 41)
    stream = torch.cuda.current_stream()
    want = G.oracle_expected(sh, a, b, "bf16", "bf16", False, [s.cpu().numpy() for s in src])
    for _ in range(2):
        mid = G.Guarded([t.buffer_bytes(True, j) for j in range(4)])
        back = G.Guarded([t.buffer_bytes(True, 4 + j) for j in range(4)])
        t.run_static([s.data_ptr() for s in src], mid.ptrs() + back.ptrs(), stream.cuda_stream)
        stream.synchronize()
        assert B.static_status() == B.DEV_OK
        for g, w in zip(mid.bufs, want):
            assert np.array_equal(g.cpu().numpy(), w)
        for g, s in zip(back.bufs, src):
            assert torch.equal(g, s)                                     # the round trip restores the source bits
        assert mid.guards_intact() and back.guards_intact()
    monkeypatch.setenv("NEREUS_DEBUG_GATE_BIAS", "1000000")
    mid = G.Guarded([t.buffer_bytes(True, j) for j in range(4)])
    back = G.Guarded([t.buffer_bytes(True, 4 + j) for j in range(4)])
    t.run_static([s.data_ptr() for s in src], mid.ptrs() + back.ptrs(), stream.cuda_stream)
    stream.synchronize()                                                 # returns: the wait is bounded
    monkeypatch.delenv("NEREUS_DEBUG_GATE_BIAS")
    assert t.status() == B.DEV_OK                                        # the handle's own status word is untouched
    assert B.static_status() == B.DEV_TIMEOUT
    assert B.static_status() == B.DEV_OK                                 # reading it cleared it
    for r in back.raw:
        assert bool((r == G.SENTINEL).all())                             # nothing of level 1 was written
    t.run_static([s.data_ptr() for s in src], mid.ptrs() + back.ptrs(), stream.cuda_stream)
    stream.synchronize()
    assert B.static_status() == B.DEV_OK
    for g, s in zip(back.bufs, src):
        assert torch.equal(g, s)


def test_run_static_leaves_device_memory_alone_and_refuses_capture():
    desc, t, src, sizes = _pair(*CASES[0])
    out = G.Guarded(sizes)
    stream = torch.cuda.Stream()
    sp, dp = [s.data_ptr() for s in src], out.ptrs()
    t.run_static(sp, dp, stream.cuda_stream)                             # any first-call set-up happens here
    stream.synchronize()
    free0, _ = torch.cuda.mem_get_info()
    for _ in range(3):
        t.run_static(sp, dp, stream.cuda_stream)
    stream.synchronize()
    free1, _ = torch.cuda.mem_get_info()
    assert free1 == free0                                                # nothing was taken from the device
    # while the stream is being captured the upload from the shared host arrays would be replayed stale
    g = torch.cuda.CUDAGraph()
    with torch.cuda.graph(g, stream=stream):
        rc = t.run_static_raw(sp, dp, stream.cuda_stream)
    assert rc == B.ERR_UNSUPPORTED
    t.run_static(sp, dp, stream.cuda_stream)                             # and works again afterwards
    stream.synchronize()
    assert B.static_status() == B.DEV_OK
    _assert_equals_oracle(CASES[0], src, out)


def test_run_static_refuses_what_does_not_fit_or_does_not_validate():
    sh = I.Shape(128, 64, 8, 8, 128, 128)                                # 128 layers x 8 ranks: > 4096 tasks
    desc = G.desc_of(sh)
    t = desc.compile(B.Plan(1, 1), B.Plan(8, 1))
    assert len(t.rects()) > B.STATIC_MAX_RECTS
    src = G.device_sources(desc, B.Plan(1, 1), "bf16", 1)
    out = G.Guarded([t.buffer_bytes(True, j) for j in range(8)])
    assert t.run_static_raw([s.data_ptr() for s in src], out.ptrs()) == B.ERR_TOO_LARGE
    assert "fixed scratch" in B.strerror(B.ERR_TOO_LARGE)
    G.run_transition(t, src, out.bufs)                                   # the allocating entry point takes it
    # a task that leaves its buffer is refused by the host-side check, before anything is enqueued
    desc, t, src, sizes = _pair(*CASES[0])
    bad = t.rects()[0]
    bad.dst_off = sizes[bad.dst_buf - 1] - 16
    t.debug_set_rect(0, bad)
    out = G.Guarded(sizes)
    assert t.run_static_raw([s.data_ptr() for s in src], out.ptrs()) == B.ERR_TABLE
    torch.cuda.synchronize()
    for r in out.raw:
        assert bool((r == G.SENTINEL).all())
