"""Host logic of the CUDA library, checked without a GPU: exported symbols, layout queries, and the
transition compiler's task table executed by a byte-loop interpreter (test scaffolding only) against the
oracle."""
import itertools
import os
import re

import numpy as np
import pytest

from oracle import oracle as O
from paper_2609_34645_b200 import binding as B
from paper_2609_34645_b200 import inputs as I

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def desc_of(sh, dtype=B.BF16, value_head=False):
    return B.ModelDesc(sh.layers, sh.hidden, sh.heads, sh.kv_heads, sh.ffn, sh.vocab, dtype, value_head)


def omodel_of(sh, dtype=O.BF16, value_head=False):
    return O.Model(sh.layers, sh.hidden, sh.heads, sh.kv_heads, sh.ffn, sh.vocab, dtype, value_head)


def random_src(m, plan, seed, dtype):
    """Seeded N(0, 0.02) source shards with replicated tensors tied, laid out by the oracle's layout."""
    sizes = [O.shard_bytes(m, plan, s) for s in range(O.num_shards(m, plan))]
    bufs = I.make_shards(sizes, dtype, seed)
    groups = []
    for t in range(O.num_logical(m)):
        same = {}                                    # parts that cover the same region are copies of each other
        for s in range(len(sizes)):
            p = O.locate(m, plan, s, t)
            if p.held:
                same.setdefault((p.r0, p.c0, p.nr, p.nc), []).append((s, p.offset, p.nr * p.nc * O.es(m, plan)))
        groups += [g for g in same.values() if len(g) > 1]
    I.tie_replicas(bufs, groups)
    return [b.numpy() for b in bufs]


def interpret(rects, src, dst, counts=None):
    """Executes rect tasks on host byte arrays, level by level, in table order."""
    bufs = list(src) + list(dst)
    for r in rects:
        s = bufs[r.src_buf]
        for i in range(r.rows):
            so, do = r.src_off + i * r.src_pitch, r.dst_off + i * r.dst_pitch
            piece = s[so:so + r.width_bytes_src]
            if r.cast:
                piece = O.rne_bf16_array(piece.view(np.uint32)).view(np.uint8)
            assert piece.size == r.width_bytes_dst
            for j in range(r.replicas):
                k = r.dst_buf + j * r.replica_stride
                bufs[k][do:do + r.width_bytes_dst] = piece
                if counts is not None:
                    counts[k - len(src)][do:do + r.width_bytes_dst] += 1


def payload_mask(m, plan):
    masks = [np.zeros(O.shard_bytes(m, plan, s), bool) for s in range(O.num_shards(m, plan))]
    e = O.es(m, plan)
    for s in range(len(masks)):
        for t in range(O.num_logical(m)):
            p = O.locate(m, plan, s, t)
            if p.held:
                masks[s][p.offset:p.offset + p.nr * p.nc * e] = True
    return masks


def plans_for(sh):
    return [(tp, pp) for tp in (1, 2, 4, 8) for pp in (1, 2, 4, 8)
            if tp <= sh.kv_heads and sh.kv_heads % tp == 0 and sh.ffn % tp == 0 and sh.vocab % tp == 0
            and sh.layers % pp == 0]


# ---------------------------------------------------------------- the boundary

def test_library_exports_every_declared_symbol():
    with open(os.path.join(ROOT, "include", "nereus.h")) as f:
        text = re.sub(r"/\*.*?\*/", "", f.read(), flags=re.S)
    declared = set(re.findall(r"\b(nereus_[a-z_0-9]+)\s*\(", text))
    assert declared, "no declarations found"
    assert declared == set(B.EXPORTS)
    import ctypes
    lib = ctypes.CDLL(B.LIB_PATH)
    for name in declared:
        assert hasattr(lib, name), name


def test_argument_errors():
    d = desc_of(I.TINY)
    assert d.plan_check(B.Plan(4, 1)) == B.OK                      # tp > kv_heads: kv heads are replicated
    assert d.plan_check(B.Plan(8, 1)) == B.ERR_INDIVISIBLE         # more ranks than q heads
    assert d.plan_check(B.Plan(1, 4)) == B.ERR_INDIVISIBLE         # 2 layers over 4 stages
    assert d.plan_check(B.Plan(0, 1)) == B.ERR_ARG
    assert d.plan_check(B.Plan(1, 1, 7)) == B.ERR_ARG
    with pytest.raises(B.NereusError) as e:
        B.ModelDesc(2, 256, 3, 2, 688, 1024)
    assert e.value.code == B.ERR_INDIVISIBLE
    with pytest.raises(B.NereusError) as e:
        B.ModelDesc(0, 256, 4, 2, 688, 1024)
    assert e.value.code == B.ERR_ARG
    with pytest.raises(B.NereusError) as e:
        d.compile(B.Plan(1, 1, B.BF16), B.Plan(1, 1, B.FP32))      # bf16 -> fp32 is not a transition
    assert e.value.code == B.ERR_UNSUPPORTED
    with pytest.raises(B.NereusError) as e:
        d.set_value_head(2)
    assert e.value.code == B.ERR_UNSUPPORTED
    # F/tp = 86 elements = 172 bytes: not a multiple of 16
    with pytest.raises(B.NereusError) as e:
        desc_of(I.Shape(2, 256, 4, 2, 172, 1024)).compile(B.Plan(1, 1), B.Plan(2, 1))
    assert e.value.code == B.ERR_INDIVISIBLE
    assert "16 bytes" in B.strerror(B.ERR_INDIVISIBLE)


# ---------------------------------------------------------------- layout

@pytest.mark.parametrize("sh,vh", [(I.TINY, False), (I.MICRO, True), (I.LLAMA_8B, False), (I.LLAMA_8B, True),
                                   (I.DENSE_32B, False)])
def test_layout_agrees_with_oracle(sh, vh):
    """Shard sizes and every stored tensor's offset and extent equal the oracle's independent derivation."""
    for es, bdt, odt in ((2, B.BF16, O.BF16), (4, B.FP32, O.FP32)):
        d, m = desc_of(sh, bdt, vh), omodel_of(sh, odt, vh)
        L = sh.layers
        assert d.num_tensors() == 6 * L + 3
        pls = plans_for(sh) if sh.layers <= 8 else [(1, 1), (4, 2), (2, 2), (4, 1), (8, 1), (2, 4)]
        pls = [p for p in pls if p in plans_for(sh)]
        for tp, pp in pls:
            bp, op = B.Plan(tp, pp), O.Plan(tp, pp)
            assert d.num_shards(bp) == O.num_shards(m, op)
            layers = range(L) if L <= 8 else (0, 1, L // 2 - 1, L // 2, L - 1)
            for s in range(tp * pp):
                assert d.shard_bytes(bp, s) == O.shard_bytes(m, op, s)
                # stored id -> the oracle's logical ids that make it up
                pairs = [(0, [0]), (1 + 6 * L, [9 * L + 1]), (2 + 6 * L, [9 * L + 2])]
                for l in layers:
                    b6, b9 = 1 + 6 * l, 1 + 9 * l
                    pairs += [(b6, [b9]), (b6 + 1, [b9 + 1, b9 + 2, b9 + 3]), (b6 + 2, [b9 + 4]), (b6 + 3, [b9 + 5]),
                              (b6 + 4, [b9 + 6, b9 + 7]), (b6 + 5, [b9 + 8])]
                for sid, lids in pairs:
                    off, rows, cols, rep = d.tensor_slice(bp, s, sid)
                    parts = [O.locate(m, op, s, t) for t in lids]
                    if not parts[0].held:
                        assert rows == 0 and cols == 0
                        continue
                    assert off == parts[0].offset
                    assert rows * cols == sum(p.nr * p.nc for p in parts)
                    assert cols == parts[0].nc
                    cur = off
                    for p in parts:                      # fused parts are stacked back to back
                        assert p.offset == cur
                        cur += p.nr * p.nc * es


# ---------------------------------------------------------------- the compiler, executed on the host

def check_transition(sh, a, b, sdt="bf16", ddt="bf16", vh=False, seed=0, la=0, lb=0):
    odt = {"bf16": O.BF16, "fp32": O.FP32}
    d = desc_of(sh, B.DTYPES[sdt], vh)
    m = omodel_of(sh, odt[sdt], vh)
    oa, ob = O.Plan(a[0], a[1], 0, la), O.Plan(b[0], b[1], odt[ddt], lb)
    src = random_src(m, oa, seed, sdt)
    want = O.reshard(m, oa, ob, src, fill=0xA5)
    t = d.compile(B.Plan(a[0], a[1], 0, la), B.Plan(b[0], b[1], B.DTYPES[ddt], lb))
    assert t.validate() == B.OK                      # what the compiler emits passes the host-side table check
    n_src, n_dst = t.num_buffers()
    assert (n_src, n_dst) == (len(src), len(want))
    for i, s in enumerate(src):
        assert t.buffer_bytes(False, i) == s.size
    got = [np.full(t.buffer_bytes(True, j), 0xA5, np.uint8) for j in range(n_dst)]
    counts = [np.zeros(g.size, np.uint8) for g in got]
    rects = t.rects()
    interpret(rects, src, got, counts)
    m_dst = omodel_of(sh, odt[ddt], vh)
    for j, (g, w, c, mask) in enumerate(zip(got, want, counts, payload_mask(m_dst, O.Plan(b[0], b[1], 0, lb & 4)))):
        assert np.array_equal(g, w), (a, b, j)
        assert np.array_equal(c == 1, mask), "every payload byte written exactly once, padding never"
    rd, wr = t.bytes()
    assert wr == sum(int(mk.sum()) for mk in payload_mask(m_dst, O.Plan(b[0], b[1], 0, lb & 4)))
    assert rd == wr * (2 if sdt != ddt else 1)
    for r in rects:
        assert r.src_off % 16 == 0 and r.dst_off % 16 == 0 and r.width_bytes_dst % 16 == 0
        if r.rows > 1:
            assert r.src_pitch % 16 == 0 and r.dst_pitch % 16 == 0
    return t


@pytest.mark.parametrize("a,b", list(itertools.product([(1, 1), (2, 1), (1, 2), (2, 2)], repeat=2)))
def test_tiny_all_plan_pairs(a, b):
    check_transition(I.TINY, a, b)


def test_micro_plan_pairs_including_paper_example():
    pls = plans_for(I.MICRO)
    rng = np.random.default_rng(0)
    pairs = [((4, 8), (8, 2)), ((4, 8), (4, 2)), ((4, 2), (8, 2)), ((1, 4), (2, 4)), ((8, 1), (1, 8))]
    pairs += [(pls[i], pls[j]) for i, j in rng.integers(0, len(pls), (12, 2))]
    for a, b in pairs:
        check_transition(I.MICRO, a, b, seed=3)


@pytest.mark.parametrize("a,b", [((2, 2), (4, 1)), ((1, 1), (2, 2)), ((4, 4), (1, 1)), ((2, 1), (2, 1))])
def test_cast_transitions(a, b):
    check_transition(I.SMALL, a, b, "fp32", "bf16", seed=2)


@pytest.mark.parametrize("la,lb", [(la, lb) for la in range(4) for lb in range(4) if la or lb])
def test_layout_variants(la, lb):
    """Grouped QKV and row-interleaved gate/up on either side, with TP and PP changing at the same time."""
    check_transition(I.SMALL, (2, 2), (4, 1), seed=la * 4 + lb, la=la, lb=lb)
    check_transition(I.MICRO, (8, 1), (2, 4), seed=5, la=la, lb=lb)
    check_transition(I.TINY, (1, 1), (2, 1), "fp32", "bf16", seed=6, la=la, lb=lb)


def test_layout_variant_task_shapes():
    d = desc_of(I.LLAMA_8B, B.FP32)
    t = d.compile(B.Plan(2, 2, 0, 3), B.Plan(4, 1, B.BF16, 0))
    rects = t.rects()
    pitched = {(r.rows, r.width_bytes_dst, r.src_pitch) for r in rects if r.rows > 1 and r.width_bytes_dst == 8192}
    assert pitched == {(14336 // 4, 8192, 32768)}             # gate / up rows picked out of the interleaved source
    assert d.plan_check(B.Plan(2, 2, 0, 8)) == B.ERR_ARG       # unknown layout flag
    same = d.compile(B.Plan(2, 2, 0, 3), B.Plan(2, 2, 0, 3))
    assert all(r.rows == 1 for r in same.rects())              # same layout on both sides: runs only


GQA16 = I.Shape(2, 128, 16, 2, 256, 256)          # 16 q heads, 2 kv heads, head_dim 8: room for tp up to 16


@pytest.mark.parametrize("a,b", [((1, 1), (8, 1)), ((8, 2), (2, 1)), ((16, 1), (4, 2)), ((4, 1), (16, 1)),
                                 ((8, 1), (8, 2)), ((2, 2), (16, 1))])
def test_kv_head_replication(a, b):
    """tp > kv_heads on either side: replicated kv heads are written to every rank that needs them and read
    from the first rank that has them; with the cast and with grouped QKV as well."""
    check_transition(GQA16, a, b, seed=1)
    check_transition(GQA16, a, b, "fp32", "bf16", seed=2, la=1, lb=0)
    check_transition(GQA16, a, b, seed=3, la=3, lb=3)


def test_non_nested_degrees():
    """The primitives allow any integer ratio between compatible layouts, not only powers of two (Section 5.2): TP 3 <-> 2
    <-> 6 and PP 3 <-> 1, where destination slices straddle source slices."""
    sh = I.Shape(3, 192, 6, 6, 384, 768)                       # 6 q heads, 6 kv heads, head_dim 32
    for a, b in [((3, 1), (2, 3)), ((2, 3), (3, 1)), ((6, 1), (2, 1)), ((1, 3), (6, 1)), ((3, 3), (2, 1))]:
        check_transition(sh, a, b, seed=4)
        check_transition(sh, a, b, "fp32", "bf16", seed=5, la=1, lb=2)


def test_padded_vocabulary():
    """NEREUS_VOCAB_PADDED on either side: padding rows take room, are never read and never written; a vocabulary
    that tp does not divide can only be cut this way."""
    sh = I.Shape(2, 64, 4, 4, 128, 1000)
    for (a, la), (b, lb) in [(((1, 1), 0), ((4, 2), 4)), (((4, 2), 4), ((1, 1), 0)), (((2, 1), 4), ((4, 1), 4)),
                             (((4, 1), 4), ((2, 2), 0)), (((2, 2), 5), ((4, 1), 6)), (((2, 1), 4), ((2, 1), 4))]:
        check_transition(sh, a, b, seed=7, la=la, lb=lb)
        check_transition(sh, a, b, "fp32", "bf16", seed=8, la=la, lb=lb)
    odd = I.Shape(2, 64, 4, 4, 128, 1001)
    d = desc_of(odd)
    assert d.plan_check(B.Plan(2, 1)) == B.ERR_INDIVISIBLE and d.plan_check(B.Plan(2, 1, 0, 4)) == B.OK
    check_transition(odd, (1, 1), (4, 1), seed=9, la=0, lb=4)
    d8 = desc_of(I.Shape(2, 64, 4, 4, 128, 1000))
    assert d8.shard_bytes(B.Plan(4, 1, 0, 4), 0) > d8.shard_bytes(B.Plan(4, 1), 0)


def test_uneven_pipeline_cut():
    """pp that does not divide the layer count, on either side."""
    sh = I.Shape(7, 64, 4, 4, 128, 256)
    for a, b in [((1, 1), (2, 3)), ((2, 3), (4, 4)), ((4, 4), (1, 7)), ((2, 5), (2, 2)), ((1, 7), (1, 3))]:
        check_transition(sh, a, b, seed=11)
        check_transition(sh, a, b, "fp32", "bf16", seed=12, la=3, lb=0)


def test_value_head_and_fp32():
    check_transition(I.SMALL, (2, 1), (4, 2), vh=True, seed=5)
    check_transition(I.SMALL, (4, 1), (2, 1), vh=True, seed=7)
    check_transition(I.TINY, (1, 1), (2, 2), "fp32", "fp32", seed=1)


def test_rect_counts_and_bytes_closed_form_8b():
    d = desc_of(I.LLAMA_8B)
    t = d.compile(B.Plan(1, 1), B.Plan(4, 2))
    rd, wr = t.bytes()
    repl = (2 * 32 + 1) * 4096 * 2 * 3                 # norms written once per extra TP replica
    assert rd == wr == 8_030_261_248 * 2 + repl
    rects = t.rects()
    assert all(r.level == 0 and r.cast == 0 for r in rects)
    sizes = [r.rows * r.width_bytes_dst for r in rects]
    assert sizes == sorted(sizes, reverse=True)        # largest first
    pitched = [r for r in rects if r.rows > 1]
    assert len(pitched) == 32 * 4 * 2                  # wo and wdown, per layer and destination rank
    assert {r.width_bytes_dst for r in pitched} == {2048, 7168}
    t3 = desc_of(I.LLAMA_8B, B.FP32).compile(B.Plan(2, 2), B.Plan(4, 1, B.BF16))
    rd, wr = t3.bytes()
    assert rd == 2 * wr and wr == 8_030_261_248 * 2 + repl
    assert all(r.cast == 1 for r in t3.rects())


def test_identity_collapses_to_runs():
    """Equal plans: every task is a contiguous run, adjacent tensors merged where no padding separates them."""
    t = desc_of(I.TINY).compile(B.Plan(2, 1), B.Plan(2, 1))
    assert all(r.rows == 1 for r in t.rects())


def test_tiles_cover_tasks():
    t = desc_of(I.SMALL).compile(B.Plan(1, 1), B.Plan(4, 2))
    for tile in (512, 4096, 16384, 1 << 20):
        t.tune(tile_bytes=tile)
        tiles, levels = t.num_tiles()
        want = 0
        for r in t.rects():
            if r.rows == 1 or r.width_bytes_dst >= tile:
                want += r.rows * -(-r.width_bytes_dst // tile)
            else:
                want += -(-r.rows // max(1, tile // r.width_bytes_dst))
        assert tiles == want and levels == 1
    with pytest.raises(B.NereusError):
        t.tune(tile_bytes=1000)


@pytest.mark.parametrize("kind", ["split", "merge_cast", "layouts_replicated", "chained"])
@pytest.mark.parametrize("tune", [dict(), dict(tile_bytes=512), dict(tile_bytes=1536, variant=1),
                                  dict(tile_bytes=4096, variant=2), dict(tile_bytes=65536, variant=3)])
def test_tiles_executed_one_by_one_equal_the_oracle(kind, tune):
    """What the kernels walk: every tile of the tiling, executed on host bytes as the small task it amounts to,
    in claim order.  The result must equal the oracle's, every payload byte written exactly once, and the tiles
    must be the tasks cut up (same buffers, level, cast; levels in order)."""
    sh = I.SMALL
    if kind == "split":
        d, m = desc_of(sh), omodel_of(sh)
        oa, ob, k = O.Plan(1, 1), O.Plan(4, 2), 1
        t = d.compile(B.Plan(1, 1), B.Plan(4, 2))
    elif kind == "merge_cast":
        d, m = desc_of(sh, B.FP32), omodel_of(sh, O.FP32)
        oa, ob, k = O.Plan(4, 2), O.Plan(2, 1, O.BF16), 1
        t = d.compile(B.Plan(4, 2), B.Plan(2, 1, B.BF16))
    elif kind == "layouts_replicated":
        d, m = desc_of(sh), omodel_of(sh)
        oa, ob, k = O.Plan(2, 2, 0, 3), O.Plan(4, 1, 0, 0), 2
        t = d.compile_replicated(B.Plan(2, 2, 0, 3), B.Plan(4, 1, 0, 0), 2)
    else:
        d, m = desc_of(sh), omodel_of(sh)
        oa, ob, k = O.Plan(2, 2), O.Plan(4, 1), 1
        t = B.Transition.fuse([d.compile(B.Plan(2, 2), B.Plan(4, 1)), d.compile(B.Plan(4, 1), B.Plan(2, 2))], chained=True)
    t.tune(**tune)
    src = random_src(m, oa, 17, "fp32" if kind == "merge_cast" else "bf16")
    n_src, n_dst = t.num_buffers()
    got = [np.full(t.buffer_bytes(True, j), 0xA5, np.uint8) for j in range(n_dst)]
    counts = [np.zeros(g.size, np.uint8) for g in got]
    tiles = t.tiles()
    assert len(tiles) == t.num_tiles()[0]
    assert [x.level for x in tiles] == sorted(x.level for x in tiles)
    assert sum(x.rows * x.width_bytes_dst * x.replicas for x in tiles) == t.bytes()[1]
    tile_bytes = t.launch_info()["tile_bytes"]
    assert all(x.rows * x.width_bytes_dst <= max(tile_bytes, x.width_bytes_dst) for x in tiles)
    assert t.tiles(3, 2)[0].dst_off == tiles[3].dst_off and len(t.tiles(len(tiles), 0)) == 0
    interpret(tiles, src, got, counts)
    want = O.reshard_replicated(m, oa, ob, k, src, fill=0xA5)
    for g, w in zip(got, want):
        assert np.array_equal(g, w)
    if kind == "chained":
        for mk, g, s_ in zip(payload_mask(m, oa), got[4:], src):
            assert np.array_equal(g[mk], s_[mk])
    m_dst = omodel_of(sh, O.BF16) if kind == "merge_cast" else m
    for j, mask in enumerate(payload_mask(m_dst, O.Plan(ob.tp, ob.pp)) * k):
        assert np.array_equal(counts[j] == 1, mask), "every payload byte written exactly once, padding never"


# ---------------------------------------------------------------- fuse

def test_fuse_independent_and_chained():
    sh = I.TINY
    d, m = desc_of(sh), omodel_of(sh)
    a, b = (2, 1), (1, 2)
    t_ab = d.compile(B.Plan(*a), B.Plan(*b))
    t_ba = d.compile(B.Plan(*b), B.Plan(*a))
    src = random_src(m, O.Plan(*a), 4, "bf16")
    mid_want = O.reshard(m, O.Plan(*a), O.Plan(*b), src, fill=0xA5)

    # chained round trip: level 0 writes `mid`, level 1 reads it and writes `back`
    ch = B.Transition.fuse([t_ab, t_ba], chained=True)
    assert ch.validate() == B.OK
    assert ch.num_buffers() == (2, 4)
    assert ch.num_tiles()[1] == 2
    rects = ch.rects()
    assert [r.level for r in rects] == sorted(r.level for r in rects)
    mid = [np.full(ch.buffer_bytes(True, j), 0xA5, np.uint8) for j in range(2)]
    back = [np.full(ch.buffer_bytes(True, 2 + j), 0xA5, np.uint8) for j in range(2)]
    interpret(rects, src, mid + back)
    for g, w in zip(mid, mid_want):
        assert np.array_equal(g, w)
    for mk, g, s in zip(payload_mask(m, O.Plan(*a)), back, src):
        assert np.array_equal(g[mk], s[mk])
    rd, wr = ch.bytes()
    assert rd == wr == sum(t_ab.bytes()[1:]) + sum(t_ba.bytes()[1:])

    # independent: two model-stages side by side
    ind = B.Transition.fuse([t_ab, t_ba], chained=False)
    assert ind.validate() == B.OK
    assert ind.num_buffers() == (4, 4)
    src2 = random_src(m, O.Plan(*b), 6, "bf16")
    out = [np.full(ind.buffer_bytes(True, j), 0xA5, np.uint8) for j in range(4)]
    interpret(ind.rects(), src + src2, out)
    for g, w in zip(out, mid_want + O.reshard(m, O.Plan(*b), O.Plan(*a), src2, fill=0xA5)):
        assert np.array_equal(g, w)

    # parts that do not connect
    with pytest.raises(B.NereusError) as e:
        B.Transition.fuse([t_ab, t_ab], chained=True)
    assert e.value.code == B.ERR_MISMATCH
    with pytest.raises(B.NereusError) as e:
        B.Transition.fuse([ch, t_ab], chained=False)          # only compiled parts fuse
    assert e.value.code == B.ERR_ARG


def test_run_rejects_bad_pointers_before_any_cuda_call():
    t = desc_of(I.TINY).compile(B.Plan(2, 1), B.Plan(1, 1))
    sizes = [t.buffer_bytes(False, 0), t.buffer_bytes(False, 1)]
    base = 1 << 40
    src = [base, base + (1 << 30)]
    assert t.run_raw([0, src[1]], [base + (2 << 30)]) == B.ERR_ARG
    assert t.run_raw([src[0] + 8, src[1]], [base + (2 << 30)]) == B.ERR_ALIGN
    assert t.run_raw(src, [src[1] + sizes[1] - 256]) == B.ERR_ALIAS        # dst overlaps a source's tail
    assert t.run_raw(src, [src[0] - 16]) == B.ERR_ALIAS
    # declared lengths: a buffer shorter than required is refused, before any CUDA call as well
    dst, need = [base + (2 << 30)], [t.buffer_bytes(True, 0)]
    assert t.run_sized_raw(src, [sizes[0], sizes[1] - 1], dst, need) == B.ERR_TOO_SMALL
    assert t.run_sized_raw(src, sizes, dst, [need[0] - 256]) == B.ERR_TOO_SMALL
    assert t.run_sized_raw([0, src[1]], sizes, dst, need) == B.ERR_ARG            # then run()'s own checks
    assert "shorter" in B.strerror(B.ERR_TOO_SMALL)
    # the per-block trace: nothing to read before a traced run has been prepared
    t.trace(True)
    with pytest.raises(B.NereusError) as e:
        t.trace_read()
    assert e.value.code == B.ERR_ARG
    t.trace(False)


# ---------------------------------------------------------------- replicas (Extend) and optimizer state

@pytest.mark.parametrize("a,b,k,sdt,ddt", [((2, 2), (2, 2), 3, "bf16", "bf16"),      # Extend: same layout, 3 new units
                                           ((4, 1), (2, 2), 2, "bf16", "bf16"),      # Split into 2 replica units
                                           ((2, 2), (4, 1), 2, "fp32", "bf16")])     # weight sync to 2 rollout units
def test_replicated_destinations(a, b, k, sdt, ddt):
    sh = I.SMALL
    odt = {"bf16": O.BF16, "fp32": O.FP32}
    d, m = desc_of(sh, B.DTYPES[sdt]), omodel_of(sh, odt[sdt])
    src = random_src(m, O.Plan(*a), 11, sdt)
    want = O.reshard_replicated(m, O.Plan(*a), O.Plan(b[0], b[1], odt[ddt]), k, src, fill=0xA5)
    t = d.compile_replicated(B.Plan(*a), B.Plan(b[0], b[1], B.DTYPES[ddt]), k)
    n_src, n_dst = t.num_buffers()
    assert n_dst == k * b[0] * b[1] == len(want)
    got = [np.full(t.buffer_bytes(True, j), 0xA5, np.uint8) for j in range(n_dst)]
    counts = [np.zeros(g.size, np.uint8) for g in got]
    interpret(t.rects(), src, got, counts)
    for g, w in zip(got, want):
        assert np.array_equal(g, w)
    rd, wr = t.bytes()
    one = d.compile(B.Plan(*a), B.Plan(b[0], b[1], B.DTYPES[ddt])).bytes()
    assert rd == one[0] and wr == k * one[1]          # read once, written k times
    if a == b and sdt == ddt:                          # Extend: every unit is a copy of the source unit
        masks = payload_mask(m, O.Plan(*a))
        for j, g in enumerate(got):
            mk = masks[j % len(src)]
            assert np.array_equal(g[mk], src[j % len(src)][mk])
    with pytest.raises(B.NereusError) as e:
        d.compile_replicated(B.Plan(*a), B.Plan(*b), 0)
    assert e.value.code == B.ERR_ARG


def test_state_with_optimizer_tensors():
    """theta (bf16) plus Adam's two fp32 moments, all following the same layout, in one table."""
    sh = I.SMALL
    d, m = desc_of(sh), omodel_of(sh)
    a, b = (2, 2), (4, 1)
    m32 = omodel_of(sh, O.FP32)
    src = random_src(m, O.Plan(*a), 1, "bf16") + random_src(m32, O.Plan(*a), 2, "fp32") + \
        random_src(m32, O.Plan(*a), 3, "fp32")
    want = O.reshard_state(m, O.Plan(*a), O.Plan(*b), 2, src, fill=0xA5)
    t = d.compile_state(B.Plan(*a), B.Plan(*b), 2)
    assert t.num_buffers() == (12, 12)
    got = [np.full(t.buffer_bytes(True, j), 0xA5, np.uint8) for j in range(12)]
    interpret(t.rects(), src, got)
    for g, w in zip(got, want):
        assert np.array_equal(g, w)
    rd, wr = t.bytes()
    theta = d.compile(B.Plan(*a), B.Plan(*b)).bytes()[0]
    assert rd == wr == theta * (1 + 2 * 2)            # fp32 moments are twice the bf16 parameters, each


def test_launch_shapes_without_a_device():
    """launch_info before prepare answers for a 148-SM device: the default kernel by table, and forced kernels on
    tables they were not made for (a tiny cast table through the ring: the halved default tile must stay a
    multiple of 512 bytes)."""
    d32 = desc_of(I.Shape(1, 64, 4, 2, 64, 64), B.FP32)
    t = d32.compile(B.Plan(2, 1), B.Plan(1, 1, B.BF16))
    assert t.launch_info()["kernel"] == "nereus_walk_once" and t.launch_info()["tile_bytes"] == 1024
    t.tune(variant=2)
    li = t.launch_info()
    assert li["kernel"] == "nereus_walk_ring" and li["tile_bytes"] % 512 == 0 and li["tile_bytes"] >= 1024
    assert li["threads"] == 512 and li["grid"] == 148             # the converting ring: 1 + 15 warps, one CTA per SM
    t.tune(variant=1)
    assert t.launch_info()["kernel"] == "nereus_walk_vec" and t.launch_info()["tile_bytes"] % 512 == 0
    big = desc_of(I.LLAMA_8B).compile(B.Plan(1, 1), B.Plan(4, 2))
    li = big.launch_info()
    assert (li["kernel"], li["tile_bytes"], li["grid"], li["threads"]) == ("nereus_walk_ring", 32768, 148, 64)
    assert big.num_tiles() == (506756, 1)
    # 512-byte row pieces (wo at TP16) in 8% of the bytes: the large table goes to the vector kernel
    tp16 = desc_of(I.LLAMA_8B).compile(B.Plan(4, 1), B.Plan(16, 1))
    assert tp16.launch_info()["kernel"] == "nereus_walk_vec" and tp16.launch_info()["tile_bytes"] == 16384
    assert desc_of(I.LLAMA_8B).compile(B.Plan(4, 1), B.Plan(8, 1)).launch_info()["kernel"] == "nereus_walk_ring"
    mid = desc_of(I.Shape(2, 2048, 16, 8, 5632, 8192)).compile(B.Plan(1, 1), B.Plan(4, 1))
    li = mid.launch_info()
    assert li["kernel"] == "nereus_walk_once" and li["tile_bytes"] == 4096
    assert li["grid"] == -(-mid.num_tiles()[0] // 8) and li["threads"] == 256
    mid.tune(variant=3, tile_bytes=512)                           # more tiles than get per-tile records
    assert mid.launch_info()["kernel"] == "nereus_walk_vec"
    ch = B.Transition.fuse([desc_of(I.TINY).compile(B.Plan(2, 1), B.Plan(1, 1)),
                            desc_of(I.TINY).compile(B.Plan(1, 1), B.Plan(2, 1))], chained=True)
    assert ch.launch_info()["kernel"] == "nereus_walk_vec"
    for bad in (dict(variant=4), dict(tile_bytes=700), dict(threads=100), dict(ctas_per_sm=3)):
        with pytest.raises(B.NereusError) as e:
            ch.tune(**bad)
        assert e.value.code == B.ERR_ARG


def test_buffer_limit_of_one_launch():
    """One launch addresses at most 448 buffers (its parameter block): a fused table at the limit compiles, one
    beyond it is refused; so is a single transition with more shards than that."""
    d = desc_of(I.MICRO)
    part = d.compile(B.Plan(8, 8), B.Plan(8, 4))                 # 64 + 32 buffers
    ok = B.Transition.fuse([part] * 4, chained=False)            # 384
    assert ok.num_buffers() == (256, 128)
    small = d.compile(B.Plan(8, 4), B.Plan(8, 4))                # 32 + 32
    assert B.Transition.fuse([part] * 4 + [small], chained=False).num_buffers() == (288, 160)   # 448
    with pytest.raises(B.NereusError) as e:
        B.Transition.fuse([part] * 5, chained=False)             # 480
    assert e.value.code == B.ERR_UNSUPPORTED
    with pytest.raises(B.NereusError) as e:
        d.compile_replicated(B.Plan(8, 8), B.Plan(8, 8), 7)      # 64 + 448
    assert e.value.code == B.ERR_UNSUPPORTED


def test_header_is_plain_c_and_the_library_links_from_c(tmp_path):
    """The boundary is a C ABI: nereus.h compiles as C99, and a C program that calls a few entry points links
    against the library and runs (host-only calls, no GPU needed)."""
    import subprocess
    src = tmp_path / "use_nereus.c"
    src.write_text(r'''
#include <stdio.h>
#include "nereus.h"
int main(void) {
    nereus_model_desc_t d; nereus_transition_t t; size_t rd, wr; int n;
    nereus_plan_t a = {2, 1, 0, 0}, b = {1, 1, 0, 0};
    if (nereus_model_desc(2, 256, 4, 2, 688, 1024, NEREUS_BF16, &d)) return 1;
    if (nereus_transition_compile(d, a, b, &t)) return 2;
    if (nereus_transition_bytes(t, &rd, &wr) || nereus_transition_num_rects(t, &n)) return 3;
    printf("%zu %zu %d %s\n", rd, wr, n, nereus_strerror(NEREUS_ERR_ALIAS));
    nereus_transition_destroy(t); nereus_model_desc_destroy(d);
    return 0;
}
''')
    exe = tmp_path / "use_nereus"
    libdir = os.path.dirname(B.LIB_PATH)
    subprocess.check_call(["gcc", "-std=c99", "-Wall", "-Werror", "-I", os.path.join(ROOT, "include"), str(src),
                           "-o", str(exe), "-L", libdir, "-lnereus", f"-Wl,-rpath,{libdir}"])
    out = subprocess.check_output([str(exe)], text=True).split()
    assert out[0] == out[1] == str(1_975_552 * 2) and int(out[2]) > 0


def test_binding_fails_loudly_without_the_library(tmp_path):
    """No CPU fallback: importing the binding next to no libnereus.so raises, it never degrades to something
    else."""
    import shutil
    import subprocess
    import sys
    pkg = tmp_path / "paper_2609_34645_b200"
    pkg.mkdir()
    for name in ("__init__.py", "binding.py"):
        shutil.copy(os.path.join(ROOT, "paper_2609_34645_b200", name), pkg / name)
    r = subprocess.run([sys.executable, "-c", "import paper_2609_34645_b200.binding"], cwd=tmp_path,
                       capture_output=True, text=True)
    assert r.returncode != 0 and "ImportError" in r.stderr and "no CPU fallback" in r.stderr
