"""The host-side check of the task table (nereus_transition_validate; nereus_transition_prepare and
nereus_transition_run_static run the same check before anything reaches a device): tables the compiler emits
pass, tables corrupted through the test hook are refused with NEREUS_ERR_TABLE.  No GPU needed."""

import pytest

from paper_2609_34645_b200 import binding as B
from paper_2609_34645_b200 import inputs as I


def desc_of(sh, dtype=B.BF16, value_head=False):
    return B.ModelDesc(sh.layers, sh.hidden, sh.heads, sh.kv_heads, sh.ffn, sh.vocab, dtype, value_head)


def clone(r):
    c = B.Rect()
    for name, _ in B.Rect._fields_:
        setattr(c, name, getattr(r, name))
    return c


def fresh(kind="split"):
    d = desc_of(I.SMALL)
    if kind == "split":
        return d.compile(B.Plan(1, 1), B.Plan(4, 2))
    if kind == "merge":
        return d.compile(B.Plan(4, 2), B.Plan(1, 1))
    if kind == "replicated":
        return d.compile_replicated(B.Plan(2, 2), B.Plan(4, 1), 3)
    if kind == "cast":
        return desc_of(I.SMALL, B.FP32).compile(B.Plan(2, 2), B.Plan(4, 1, B.BF16))
    if kind == "chained":
        return B.Transition.fuse([d.compile(B.Plan(2, 1), B.Plan(1, 2)), d.compile(B.Plan(1, 2), B.Plan(2, 1))],
                                 chained=True)
    raise KeyError(kind)


@pytest.mark.parametrize("kind", ["split", "merge", "replicated", "cast", "chained"])
def test_compiled_tables_pass(kind):
    assert fresh(kind).validate() == B.OK


def test_workload_tables_pass():
    """The five benchmark configurations at full size (host work only)."""
    for name in ("tiny_tp2pp1_to_tp1pp1", "8b_tp1pp1_to_tp4pp2", "8b_tp4pp2_to_tp1pp1",
                 "8b_fp32_tp2pp2_to_bf16_tp4pp1", "ppo5_8b", "32b_tp2pp4_to_tp8pp1_and_back",
                 "8b_grouped_fp32_tp2pp2_to_blocked_bf16_tp4pp1", "8b_tp4pp1_to_tp16pp1"):
        wl = I.WORKLOADS[name]
        parts = []
        for st in wl.stages:
            d = desc_of(st.shape, B.DTYPES[st.src[2]], st.value_head)
            pa = B.Plan(st.src[0], st.src[1], B.DTYPES[st.src[2]], I.layout_of(st.src))
            pb = B.Plan(st.dst[0], st.dst[1], B.DTYPES[st.dst[2]], I.layout_of(st.dst))
            parts.append(d.compile(pa, pb))
            if wl.round_trip:
                parts.append(d.compile(pb, pa))
        t = parts[0] if len(parts) == 1 else B.Transition.fuse(parts, chained=wl.round_trip)
        assert t.validate() == B.OK, name


def pitched_index(rects):
    return next(i for i, r in enumerate(rects) if r.rows > 1)


def run_index(rects):
    return next(i for i, r in enumerate(rects) if r.rows == 1 and r.width_bytes_dst >= 4096)


CORRUPTIONS = {
    # name: (table kind, function(rects, transition) -> (index, corrupted rect))
    "source offset past the end of its buffer": ("split", lambda rs, t: (0, dict(src_off=t.buffer_bytes(False, 0)))),
    "source run longer than its buffer": ("merge", lambda rs, t: (
        run_index(rs), dict(src_off=t.buffer_bytes(False, rs[run_index(rs)].src_buf) - 16))),
    "destination past the end of its buffer": ("split", lambda rs, t: (
        0, dict(dst_off=t.buffer_bytes(True, rs[0].dst_buf - t.num_buffers()[0]) - 16))),
    "last row piece of a pitched task past the end": ("split", lambda rs, t: (
        pitched_index(rs), dict(rows=rs[pitched_index(rs)].rows * 64))),
    "pitch smaller than the width": ("split", lambda rs, t: (
        pitched_index(rs), dict(dst_pitch=rs[pitched_index(rs)].width_bytes_dst - 16))),
    "source pitch smaller than the width": ("merge", lambda rs, t: (
        pitched_index(rs), dict(src_pitch=rs[pitched_index(rs)].width_bytes_src - 16))),
    "offset off the 16-byte grid": ("split", lambda rs, t: (0, dict(src_off=rs[0].src_off + 8))),
    "width off the 16-byte grid": ("split", lambda rs, t: (0, dict(width_bytes_dst=rs[0].width_bytes_dst - 8))),
    "source buffer index out of range": ("split", lambda rs, t: (0, dict(src_buf=sum(t.num_buffers())))),
    "destination index names a source": ("split", lambda rs, t: (0, dict(dst_buf=0))),
    "destination index out of range": ("split", lambda rs, t: (0, dict(dst_buf=sum(t.num_buffers())))),
    "replica lands past the last buffer": ("replicated", lambda rs, t: (0, dict(replicas=4))),
    "zero replicas": ("split", lambda rs, t: (0, dict(replicas=0))),
    "level out of range": ("split", lambda rs, t: (0, dict(level=1))),
    "levels out of execution order": ("chained", lambda rs, t: (0, dict(level=1))),
    "a task reads what its own level writes": ("chained", lambda rs, t: (
        len(rs) - 1, dict(src_buf=rs[len(rs) - 1].dst_buf))),
    "zero rows": ("split", lambda rs, t: (0, dict(rows=0))),
    "cast flag that is neither 0 nor 1": ("split", lambda rs, t: (0, dict(cast=2))),
    "two tasks write the same bytes": ("split", lambda rs, t: (
        1, dict(dst_buf=rs[0].dst_buf, dst_off=rs[0].dst_off))),
    "a run written into the rows of a pitched task": ("split", lambda rs, t: (
        run_index(rs), dict(dst_buf=rs[pitched_index(rs)].dst_buf, dst_off=rs[pitched_index(rs)].dst_off + 16,
                            width_bytes_dst=16))),
}


@pytest.mark.parametrize("what", list(CORRUPTIONS))
def test_corrupted_tables_are_refused(what):
    kind, make = CORRUPTIONS[what]
    t = fresh(kind)
    rects = t.rects()
    index, changes = make(rects, t)
    bad = clone(rects[index])
    for k, v in changes.items():
        setattr(bad, k, v)
    if "width_bytes_dst" in changes:
        bad.width_bytes_src = bad.width_bytes_dst << bad.cast
    t.debug_set_rect(index, bad)
    assert t.validate() == B.ERR_TABLE, what
    # restoring the task restores the verdict: the refusal came from that one field
    t.debug_set_rect(index, rects[index])
    assert t.validate() == B.OK


def test_column_interleaved_pieces_are_not_a_collision():
    """Row-parallel tensors gathered from several ranks interleave their row pieces in one destination block
    (bounding intervals overlap, pieces do not); shifting one of them by 16 bytes makes them collide."""
    t = desc_of(I.SMALL).compile(B.Plan(4, 1), B.Plan(1, 1))
    rects = t.rects()
    pitched = [i for i, r in enumerate(rects) if r.rows > 1]
    assert len(pitched) >= 8 and t.validate() == B.OK
    i = next(k for k in pitched if rects[k].dst_off % rects[k].dst_pitch == 0 and rects[k].rows > 1)
    bad = clone(rects[i])
    bad.dst_off += 16
    t.debug_set_rect(i, bad)
    assert t.validate() == B.ERR_TABLE


def test_hook_is_refused_once_the_table_is_on_a_device_and_checks_its_arguments():
    t = fresh()
    r = t.rects()[0]
    with pytest.raises(B.NereusError) as e:
        t.debug_set_rect(len(t.rects()), r)
    assert e.value.code == B.ERR_ARG
    assert B.strerror(B.ERR_TABLE).startswith("the task table failed validation")
