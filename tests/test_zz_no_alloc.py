"""The allocation-free entry point, nereus_transition_run_static, against nereus_transition_run.

It serves callers that cannot allocate device memory when a transition is due (their own pool owns the
GPU), so its task table lives in a fixed device array that all calls share.  The test calls it twice in a
row through the C ABI, with two different transitions so the second call must overwrite what the first one
left in the array, and asks for bit-identical destinations (the tolerance of every reshard test: none).
Collected last on purpose: a failure here stops nothing else.
"""
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


def test_run_static_matches_run_twice_in_a_row():
    assert torch.cuda.is_available()
    stream = torch.cuda.current_stream()
    cases = [_pair(I.SMALL, (1, 1), (4, 2), "bf16", "bf16", 31),        # Split, many pitched tasks
             _pair(I.SMALL, (2, 2), (4, 1), "fp32", "bf16", 32)]        # cast, a different and shorter table
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
    for want, out in zip(ref, got):
        for w, g in zip(want.raw, out.raw):                              # payload, padding and guard zones
            assert torch.equal(w, g)
    # once more in the opposite order: the first table must be restored over the second
    for (desc, t, src, sizes), want in reversed(list(zip(cases, ref))):
        out = G.Guarded(sizes)
        t.run_static([s.data_ptr() for s in src], out.ptrs(), stream.cuda_stream)
        stream.synchronize()
        for w, g in zip(want.raw, out.raw):
            assert torch.equal(w, g)


def test_run_static_refuses_what_does_not_fit():
    sh = I.Shape(128, 64, 8, 8, 128, 128)                                # 128 layers x 8 ranks: > 4096 tasks
    desc = G.desc_of(sh)
    t = desc.compile(B.Plan(1, 1), B.Plan(8, 1))
    assert len(t.rects()) > B.STATIC_MAX_RECTS
    src = G.device_sources(desc, B.Plan(1, 1), "bf16", 1)
    out = G.Guarded([t.buffer_bytes(True, j) for j in range(8)])
    assert t.run_static_raw([s.data_ptr() for s in src], out.ptrs()) == B.ERR_TOO_LARGE
    assert "fixed scratch" in B.strerror(B.ERR_TOO_LARGE)
    G.run_transition(t, src, out.bufs)                                   # the allocating entry point takes it
