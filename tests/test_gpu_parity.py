"""GPU parity: the CUDA path, called through the C ABI, against the CPU oracle, element by element on the
same seeded inputs.  Bit-exact is the bar: the reshard is a bit copy, and the cast decides a 16-bit code from
an fp32 value by one rounding rule that both sides take on the bit pattern."""
import numpy as np
import pytest
import torch

import gpu_util as G
from oracle import oracle as O
from paper_2609_34645_b200 import binding as B
from paper_2609_34645_b200 import inputs as I

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module", autouse=True)
def _need_cuda():
    assert torch.cuda.is_available(), "GPU tests need a CUDA device"


def test_tiny_merge_workload():
    """Workload 1: tiny TP2PP1 -> TP1PP1, bf16, seed 0."""
    st = I.WORKLOADS["tiny_tp2pp1_to_tp1pp1"].stages[0]
    G.check_against_oracle(st.shape, st.src[:2], st.dst[:2], st.src[2], st.dst[2], seed=st.seed)


@pytest.mark.parametrize("tile", [512, 4096, 16384, 65536])
def test_small_plan_pairs_and_tile_sizes(tile):
    """Several tiles per task and ragged tails: every nested plan pair of the SMALL shape."""
    pls = [(1, 1), (2, 1), (4, 1), (1, 2), (2, 2), (4, 2), (1, 4), (4, 4)]
    rng = np.random.default_rng(tile)
    pairs = [(pls[i], pls[j]) for i, j in rng.integers(0, len(pls), (6, 2))] + [((1, 1), (4, 2)), ((4, 2), (1, 1))]
    for a, b in pairs:
        G.check_against_oracle(I.SMALL, a, b, seed=tile, tune=dict(tile_bytes=tile, variant=1))


@pytest.mark.parametrize("tile", [512, 2048, 8192, 32768])
def test_bulk_ring_kernel(tile):
    """The bulk-copy ring (cp.async.bulk through shared memory) on the same plan pairs, incl. 16-byte pieces."""
    tune = dict(tile_bytes=tile, variant=2)
    for a, b in [((1, 1), (4, 2)), ((4, 2), (1, 1)), ((2, 4), (4, 1)), ((4, 4), (2, 2)), ((2, 1), (2, 1))]:
        G.check_against_oracle(I.SMALL, a, b, seed=tile + 1, tune=tune)
    G.check_against_oracle(I.SMALL, (2, 1), (4, 2), vh=True, seed=5, tune=tune)
    G.check_against_oracle(I.SMALL, (1, 2), (4, 1), "fp32", "fp32", seed=3, tune=tune)
    for a, b in [((4, 8), (8, 2)), ((8, 1), (1, 8))]:
        G.check_against_oracle(I.MICRO, a, b, seed=9, tune=tune)
    st = I.WORKLOADS["tiny_tp2pp1_to_tp1pp1"].stages[0]
    G.check_against_oracle(st.shape, st.src[:2], st.dst[:2], seed=0, tune=tune)
    # all-cast tables run on the ring too (consumer warps convert from shared memory); a stage holds the fp32
    # source, so the largest tile is half of a bit-copy stage
    if tile > 16384:
        return
    for a, b in [((2, 2), (4, 1)), ((1, 1), (2, 2)), ((4, 4), (1, 1)), ((2, 1), (2, 1))]:
        G.check_against_oracle(I.SMALL, a, b, "fp32", "bf16", seed=2, tune=tune)
    G.check_against_oracle(I.MICRO, (4, 8), (8, 2), "fp32", "bf16", seed=4, tune=tune)
    G.check_against_oracle(I.SMALL, (2, 2), (4, 1), "fp32", "bf16", vh=True, seed=8, tune=tune)


@pytest.mark.parametrize("tile", [512, 1536, 4096, 16384])
def test_one_warp_per_tile_kernel(tile):
    """nereus_walk_once (one warp per tile, per-tile records, no control words) on the same plan pairs: tiles of
    less than one batch, of exactly one, of several, ragged tails, 16-byte pieces, casts, value heads."""
    tune = dict(tile_bytes=tile, variant=3)
    for a, b in [((1, 1), (4, 2)), ((4, 2), (1, 1)), ((2, 4), (4, 1)), ((4, 4), (2, 2)), ((2, 1), (2, 1))]:
        t = G.check_against_oracle(I.SMALL, a, b, seed=tile + 2, tune=tune)
        assert t.launch_info()["kernel"] == "nereus_walk_once"
    G.check_against_oracle(I.SMALL, (2, 1), (4, 2), vh=True, seed=5, tune=tune)
    G.check_against_oracle(I.SMALL, (1, 2), (4, 1), "fp32", "fp32", seed=3, tune=tune)
    for a, b in [((4, 8), (8, 2)), ((8, 1), (1, 8))]:
        G.check_against_oracle(I.MICRO, a, b, seed=9, tune=tune)
    for a, b in [((2, 2), (4, 1)), ((1, 1), (2, 2)), ((4, 4), (1, 1)), ((2, 1), (2, 1))]:
        G.check_against_oracle(I.SMALL, a, b, "fp32", "bf16", seed=2, tune=tune)
    G.check_against_oracle(I.MICRO, (4, 8), (8, 2), "fp32", "bf16", seed=4, tune=tune)
    G.check_against_oracle(I.SMALL, (2, 2), (4, 1), "fp32", "bf16", vh=True, seed=8, tune=tune)
    for threads in (32, 128, 512):
        G.check_against_oracle(I.SMALL, (2, 2), (4, 1), seed=1, tune=dict(tile_bytes=tile, variant=3, threads=threads))


def test_default_kernel_by_table():
    """What runs when nothing is tuned: one warp per tile for single-level tables below 1 GiB with few buffers,
    the persistent kernels for chained tables and for tables with more buffers than its parameter block holds."""
    d = G.desc_of(I.SMALL)
    assert d.compile(B.Plan(2, 2), B.Plan(4, 1)).launch_info()["kernel"] == "nereus_walk_once"
    ch = B.Transition.fuse([d.compile(B.Plan(2, 2), B.Plan(4, 1)), d.compile(B.Plan(4, 1), B.Plan(2, 2))], chained=True)
    assert ch.launch_info()["kernel"] == "nereus_walk_vec"
    ch.tune(variant=3)                                        # asked for, not possible: falls back
    assert ch.launch_info()["kernel"] == "nereus_walk_vec"
    many = G.desc_of(I.MICRO).compile(B.Plan(8, 8), B.Plan(8, 4))          # 96 buffers
    assert many.launch_info()["kernel"] == "nereus_walk_vec"
    G.check_against_oracle(I.MICRO, (8, 8), (8, 4), seed=12)
    big = G.desc_of(I.LLAMA_8B).compile(B.Plan(1, 1), B.Plan(4, 2))
    assert big.launch_info()["kernel"] == "nereus_walk_ring"
    # a tile so small that the table has more tiles than get per-tile records: the vector kernel takes over
    t = G.desc_of(I.Shape(2, 2048, 16, 8, 5632, 8192)).compile(B.Plan(1, 1), B.Plan(4, 1))
    t.tune(variant=3, tile_bytes=512)
    assert t.num_tiles()[0] > 1 << 17 and t.launch_info()["kernel"] == "nereus_walk_vec"


@pytest.mark.parametrize("threads,ctas", [(512, 2), (256, 1), (32, 1)])
def test_launch_shapes(threads, ctas):
    G.check_against_oracle(I.SMALL, (2, 2), (4, 1), seed=1, tune=dict(threads=threads, ctas_per_sm=ctas, variant=1))
    G.check_against_oracle(I.SMALL, (2, 2), (4, 1), seed=1, tune=dict(ctas_per_sm=ctas, variant=2))


def test_micro_paper_example_and_tp8():
    """(TP4, PP8) -> (TP8, PP2), the layout example of Section 6.1, its two hops, and 16-byte row pieces."""
    for a, b in [((4, 8), (8, 2)), ((4, 8), (4, 2)), ((4, 2), (8, 2)), ((8, 1), (1, 8)), ((1, 4), (2, 4))]:
        G.check_against_oracle(I.MICRO, a, b, seed=9)


@pytest.mark.parametrize("a,b", [((2, 2), (4, 1)), ((1, 1), (2, 2)), ((4, 4), (1, 1)), ((2, 1), (2, 1))])
def test_cast_transitions(a, b):
    """fp32 -> bf16 fused into the move (the train -> generation weight sync)."""
    G.check_against_oracle(I.SMALL, a, b, "fp32", "bf16", seed=2)
    G.check_against_oracle(I.SMALL, a, b, "fp32", "bf16", seed=2, tune=dict(tile_bytes=1024))


def test_fp32_copy_and_value_head():
    G.check_against_oracle(I.SMALL, (1, 2), (4, 1), "fp32", "fp32", seed=3)
    G.check_against_oracle(I.SMALL, (2, 1), (4, 2), vh=True, seed=5)
    G.check_against_oracle(I.SMALL, (4, 1), (2, 1), vh=True, seed=7)
    G.check_against_oracle(I.SMALL, (2, 2), (4, 1), "fp32", "bf16", vh=True, seed=8)


@pytest.mark.parametrize("variant", [1, 2, 3])
def test_cast_every_fp32_bit_pattern(variant):
    """All 2^32 fp32 bit patterns through the kernel's cast (NaN, Inf, subnormals, ties) against the oracle's
    rule.  The patterns are planted in the embedding of a one-layer model, 2^28 at a time."""
    sh = I.Shape(1, 4096, 32, 8, 1024, 65536)              # embed = 2^28 elements
    desc = G.desc_of(sh, "fp32")
    pa, pb = B.Plan(1, 1), B.Plan(2, 1, B.BF16)
    t = desc.compile(pa, pb)
    t.tune(variant=variant)
    src = G.device_sources(desc, pa, "fp32", 0)
    dst = G.Guarded([t.buffer_bytes(True, j) for j in range(2)])
    off, rows, cols, _ = desc.tensor_slice(pa, 0, 0)
    n = rows * cols
    assert off == 0 and n == 1 << 28
    halves = []
    for j in range(2):
        o, r, c, _ = desc.tensor_slice(pb, j, 0)
        halves.append((o, r * c))
    ramp = torch.arange(n, dtype=torch.int64, device="cuda")
    for k in range(16):
        src[0][:4 * n].view(torch.int32).copy_((ramp + (k << 28)).to(torch.int32))   # wraps to the bit pattern
        G.run_transition(t, src, dst.bufs)
        got = torch.cat([dst.bufs[j][o:o + 2 * m] for j, (o, m) in enumerate(halves)]).cpu().numpy().view(np.uint16)
        bits = (np.arange(n, dtype=np.uint64) + (k << 28)).astype(np.uint32)
        want = O.rne_bf16_array(bits)
        assert np.array_equal(got, want), f"chunk {k}"
    assert dst.guards_intact()


def test_fused_independent_stages():
    """Five model-stages in one table (the PPO workload's structure at SMALL size, value heads included)."""
    wl = I.WORKLOADS["ppo5_8b"]
    descs, parts, srcs, wants = [], [], [], []
    for st in wl.stages:
        d = G.desc_of(I.SMALL, "bf16", st.value_head)
        pa, pb = B.Plan(*st.src[:2]), B.Plan(*st.dst[:2])
        descs.append(d)
        parts.append(d.compile(pa, pb))
        s = G.device_sources(d, pa, "bf16", st.seed)
        srcs += s
        wants += G.oracle_expected(I.SMALL, st.src[:2], st.dst[:2], "bf16", "bf16", st.value_head,
                                   [x.cpu().numpy() for x in s])
    t = B.Transition.fuse(parts, chained=False)
    n_src, n_dst = t.num_buffers()
    assert (n_src, n_dst) == (len(srcs), len(wants)) == (4 + 2 + 2 + 4 + 4, 2 + 8 + 8 + 2 + 2)
    dst = G.Guarded([t.buffer_bytes(True, j) for j in range(n_dst)])
    G.run_transition(t, srcs, dst.bufs)
    for g, w in zip(dst.bufs, wants):
        assert np.array_equal(g.cpu().numpy(), w)
    assert dst.guards_intact()
    assert t.launches() == 1


@pytest.mark.parametrize("variant", [1, 2])
@pytest.mark.parametrize("tile", [2048, 16384])
def test_chained_round_trip_into_the_sources(tile, variant):
    """A -> B -> A in one launch with dependency levels; the way back overwrites the original source
    buffers (poisoned by the test between checks), as the 32B round-trip workload does."""
    sh = I.SMALL
    d = G.desc_of(sh)
    a, b = (2, 4), (4, 1)
    ab, ba = d.compile(B.Plan(*a), B.Plan(*b)), d.compile(B.Plan(*b), B.Plan(*a))
    t = B.Transition.fuse([ab, ba], chained=True)
    t.tune(tile_bytes=tile, variant=variant)
    src = G.device_sources(d, B.Plan(*a), "bf16", 8)
    keep = [s.cpu().numpy().copy() for s in src]
    mid = G.Guarded([t.buffer_bytes(True, j) for j in range(4)])
    mid_want = G.oracle_expected(sh, a, b, "bf16", "bf16", False, keep)
    G.run_transition(t, src, mid.bufs + src)
    for g, w in zip(mid.bufs, mid_want):
        assert np.array_equal(g.cpu().numpy(), w)
    back_want = O.reshard(G.omodel_of(sh), O.Plan(*b), O.Plan(*a), mid_want, [k.copy() for k in keep])
    for g, w in zip(src, back_want):
        assert np.array_equal(g.cpu().numpy(), w)
    assert mid.guards_intact()
    # three levels: A -> B -> A -> B into fresh buffers
    t3 = B.Transition.fuse([ab, ba, ab], chained=True)
    t3.tune(tile_bytes=tile, variant=variant)
    back = G.Guarded([t3.buffer_bytes(True, 4 + j) for j in range(8)])
    again = G.Guarded([t3.buffer_bytes(True, 12 + j) for j in range(4)])
    for m in mid.bufs:
        m.fill_(G.SENTINEL)
    G.run_transition(t3, src, mid.bufs + back.bufs + again.bufs)
    for g, w in zip(again.bufs, mid_want):
        assert np.array_equal(g.cpu().numpy(), w)
    back_fresh = O.reshard(G.omodel_of(sh), O.Plan(*b), O.Plan(*a), mid_want, fill=G.SENTINEL)
    for g, w in zip(back.bufs, back_fresh):
        assert np.array_equal(g.cpu().numpy(), w)           # level 1 really wrote its fresh buffers
    assert again.guards_intact() and back.guards_intact()


def test_run_errors_on_device_pointers():
    d = G.desc_of(I.TINY)
    t = d.compile(B.Plan(2, 1), B.Plan(1, 1))
    src = G.device_sources(d, B.Plan(2, 1), "bf16", 0)
    dst = G.Guarded([t.buffer_bytes(True, 0)])
    sp = [s.data_ptr() for s in src]
    assert t.run_raw(sp, [sp[0]]) == B.ERR_ALIAS
    assert t.run_raw(sp, [dst.ptrs()[0] + 2]) == B.ERR_ALIGN
    assert t.run_raw([0, sp[1]], dst.ptrs()) == B.ERR_ARG
    assert t.launches() == 0
    # a side stream works as well as the current one
    side = torch.cuda.Stream()
    G.run_transition(t, src, dst.bufs, side)
    want = G.oracle_expected(I.TINY, (2, 1), (1, 1), "bf16", "bf16", False, [s.cpu().numpy() for s in src])
    assert np.array_equal(dst.bufs[0].cpu().numpy(), want[0])
    # chained: a destination written at level 0 may not overlap a source; at level 1 it may
    ab, ba = d.compile(B.Plan(2, 1), B.Plan(1, 1)), d.compile(B.Plan(1, 1), B.Plan(2, 1))
    ch = B.Transition.fuse([ab, ba], chained=True)
    assert ch.run_raw(sp, [sp[0]] + sp) == B.ERR_ALIAS
    assert ch.run_raw(sp, dst.ptrs() + [sp[0], sp[0]]) == B.ERR_ALIAS       # two level-1 outputs on the same memory
    assert ch.run_raw(sp, dst.ptrs() + sp) == B.OK
    torch.cuda.synchronize()
    assert ch.status() == B.DEV_OK


@pytest.mark.parametrize("variant", [1, 2])
def test_dependency_wait_gives_up_with_a_status(variant, monkeypatch):
    """Failure detection without a GPU fault: a gate that nothing will ever open (the debug bias raises its
    target) makes the bounded wait run out; the kernel returns, the host reads NEREUS_DEV_TIMEOUT, level 0 is
    complete, level 1 never wrote, and the context stays usable."""
    sh = I.SMALL
    d = G.desc_of(sh)
    a, b = (2, 2), (4, 1)
    ab, ba = d.compile(B.Plan(*a), B.Plan(*b)), d.compile(B.Plan(*b), B.Plan(*a))
    t = B.Transition.fuse([ab, ba], chained=True)
    t.tune(variant=variant)
    src = G.device_sources(d, B.Plan(*a), "bf16", 8)
    mid = G.Guarded([t.buffer_bytes(True, j) for j in range(4)])
    back = G.Guarded([t.buffer_bytes(True, 4 + j) for j in range(4)])
    stream = torch.cuda.current_stream()
    monkeypatch.setenv("NEREUS_DEBUG_GATE_BIAS", "1000000")
    t.run([s.data_ptr() for s in src], mid.ptrs() + back.ptrs(), stream.cuda_stream)
    stream.synchronize()                                       # returns: the wait is bounded
    assert t.status() == B.DEV_TIMEOUT
    want = G.oracle_expected(sh, a, b, "bf16", "bf16", False, [s.cpu().numpy() for s in src])
    for g, w in zip(mid.bufs, want):
        assert np.array_equal(g.cpu().numpy(), w)              # level 0 ran to completion
    for r in back.raw:
        assert bool((r == G.SENTINEL).all())                   # nothing of level 1 was written
    monkeypatch.delenv("NEREUS_DEBUG_GATE_BIAS")
    G.run_transition(t, src, mid.bufs + back.bufs)             # same handle, same context: works again
    for g, s in zip(back.bufs, src):
        assert torch.equal(g, s)                               # the round trip restores the source bits
    assert t.status() == B.DEV_OK
