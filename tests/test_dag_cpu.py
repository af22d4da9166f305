"""The transition-DAG planner (Section 6.1): the oracle's restatement against what the paper says in words and
figures, then the library's planner against the oracle (identical units, primitives, edges and schedule)."""
import random

import pytest

from oracle import dag as D


def U(tp, pp, first):
    return D.Unit(tp, pp, tuple(range(first, first + tp * pp)))


def ops(prims, stage=None):
    return [D.OP_NAMES[p.op] for p in prims if stage is None or p.stage == stage]


def test_t_sub_is_the_gcd_layout():
    assert D.t_sub(U(4, 8, 0), U(8, 2, 0)) == (4, 2)          # the paper's example
    assert D.t_sub(U(1, 4, 0), U(2, 4, 0)) == (1, 4)
    assert D.t_sub(U(2, 2, 0), U(2, 2, 0)) == (2, 2)


def test_reward_inference_example_of_the_dag_figure():
    """(TP4, PP8) is split into four (TP4, PP2) units, two are destroyed, the remaining two are merged into
    (TP8, PP2); actor and critic Extend onto GPUs 49-64 wait for the reward Destroys that release them."""
    S = 32 << 20                                                                       # state bytes per replica
    reward = D.StageChange(D.INFERENCE, [U(4, 8, 33)], [U(8, 2, 33)], S)               # GPUs 33..64 -> 33..48
    actor = D.StageChange(D.TRAINING, [U(4, 2, 1)], [U(4, 2, 1), U(4, 2, 49)], S)      # a replica on 49..56
    critic = D.StageChange(D.TRAINING, [U(4, 2, 9)], [U(4, 2, 9), U(4, 2, 57)], S)     # a replica on 57..64
    units, prims, order = D.plan([reward, actor, critic])
    assert ops(prims, 0) == ["split", "destroy", "destroy", "merge"]
    split = prims[0]
    assert [units[u][1:3] for u in split.dst] == [(4, 2)] * 4
    assert [units[u][3][0] for u in split.dst] == [33, 41, 49, 57]
    merge = [p for p in prims if p.op == D.MERGE][0]
    assert units[merge.dst[0]][1:3] == (8, 2) and len(merge.src) == 2
    assert ops(prims, 1) == ["extend"] and ops(prims, 2) == ["extend"]
    assert not any(p.resource_deps for p in prims)              # unlimited memory: nothing blocks
    # near capacity: a (TP4, PP2) shard is S/8; room for the split (S/32 + S/8) but not for two such shards
    units, prims, order = D.plan([reward, actor, critic], gpu_capacity=S // 8 + S // 16)
    extends = [p for p in prims if p.op == D.EXTEND]
    assert len(extends) == 2
    for p in extends:                                           # each waits for the reward Destroy on its GPUs
        assert len(p.resource_deps) == 1
        d = prims[next(iter(p.resource_deps))]
        assert d.op == D.DESTROY and d.stage == 0
        assert set(units[d.src[0]][3]) == set(units[p.dst[0]][3])
    pos = {pid: k for k, pid in enumerate(order)}
    for i, p in enumerate(prims):
        for d in p.deps | p.resource_deps:
            assert pos[d] < pos[i]                              # the schedule respects every edge


def test_emu_example_actor_tp_up_critic_dp_up():
    """Section 5.1: actor (TP1, PP4, DP2) -> (TP2, PP4, DP2) is Extend followed by Merge, DP unchanged; critic
    (TP1, PP4, DP2) -> (TP1, PP4, DP4) is two Extends."""
    actor = D.StageChange(D.GENERATION, [U(1, 4, 0), U(1, 4, 4)],
                          [D.Unit(2, 4, tuple(range(0, 4)) + tuple(range(16, 20))),
                           D.Unit(2, 4, tuple(range(4, 8)) + tuple(range(20, 24)))])
    critic = D.StageChange(D.TRAINING, [U(1, 4, 8), U(1, 4, 12)],
                           [U(1, 4, 8), U(1, 4, 12), U(1, 4, 24), U(1, 4, 28)])
    units, prims, order = D.plan([actor, critic])
    assert ops(prims, 0) == ["extend", "extend", "merge", "merge"]
    assert ops(prims, 1) == ["extend", "extend"]
    merges = [p for p in prims if p.op == D.MERGE]
    assert all(len(p.src) == 2 and units[p.dst[0]][1:3] == (2, 4) for p in merges)


def test_last_copy_is_destroyed_only_after_extend():
    """A model-stage that moves to other GPUs: its only unit is the Extend's source and is destroyed after."""
    ch = D.StageChange(D.INFERENCE, [U(2, 1, 0)], [U(2, 1, 8)])
    units, prims, order = D.plan([ch])
    assert ops(prims) == ["destroy", "extend"]
    assert 1 in prims[0].deps and order == [1, 0]


def test_infeasible_when_nothing_can_release():
    a = D.StageChange(D.GENERATION, [U(1, 1, 0)], [U(1, 1, 0), U(1, 1, 1)])
    b = D.StageChange(D.TRAINING, [U(1, 1, 1)], [U(1, 1, 1)])                     # stays: GPU 1 is never freed
    with pytest.raises(D.Infeasible):
        D.plan([a, b], gpu_capacity=1 << 20)


# ---------------------------------------------------------------- the library's planner against the oracle

from paper_2609_34645_b200 import binding as B  # noqa: E402


def lib_plan(changes, capacity=0):
    dag = B.Dag()
    for ch in changes:
        s = dag.add_stage(ch.kind, ch.state_bytes)
        for u in ch.current:
            dag.add_unit(s, False, u.tp, u.pp, list(u.gpus))
        for u in ch.target:
            dag.add_unit(s, True, u.tp, u.pp, list(u.gpus))
    dag.plan(capacity)
    return dag.units(), dag.prims()


def same_as_oracle(changes, capacity=0):
    try:
        units, prims, order = D.plan(changes, capacity or 1 << 62)
    except D.Infeasible:
        with pytest.raises(B.NereusError) as e:
            lib_plan(changes, capacity)
        assert e.value.code == B.ERR_INFEASIBLE
        return None
    lunits, lprims = lib_plan(changes, capacity)
    assert lunits == units
    assert len(lprims) == len(prims)
    for i, (a, b) in enumerate(zip(lprims, prims)):
        assert (a["op"], a["stage"], a["src"], a["dst"]) == (b.op, b.stage, b.src, b.dst), i
        assert a["deps"] == b.deps and a["resource_deps"] == b.resource_deps, i
    assert sorted(range(len(prims)), key=lambda i: lprims[i]["order"]) == order
    for a in lprims:                                   # a level is above every predecessor's
        for d in a["deps"] | a["resource_deps"]:
            assert lprims[d]["level"] < a["level"]
    return lprims


def test_library_planner_on_the_paper_examples():
    S = 32 << 20
    reward = D.StageChange(D.INFERENCE, [U(4, 8, 33)], [U(8, 2, 33)], S)
    actor = D.StageChange(D.TRAINING, [U(4, 2, 1)], [U(4, 2, 1), U(4, 2, 49)], S)
    critic = D.StageChange(D.TRAINING, [U(4, 2, 9)], [U(4, 2, 9), U(4, 2, 57)], S)
    prims = same_as_oracle([reward, actor, critic])
    assert [p["op"] for p in prims] == [B.OP_SPLIT, B.OP_DESTROY, B.OP_DESTROY, B.OP_MERGE, B.OP_EXTEND, B.OP_EXTEND]
    prims = same_as_oracle([reward, actor, critic], S // 8 + S // 16)
    assert sum(len(p["resource_deps"]) for p in prims) == 2            # the two edges of the figure
    actor2 = D.StageChange(D.GENERATION, [U(1, 4, 0), U(1, 4, 4)],
                           [D.Unit(2, 4, tuple(range(0, 4)) + tuple(range(16, 20))),
                            D.Unit(2, 4, tuple(range(4, 8)) + tuple(range(20, 24)))])
    critic2 = D.StageChange(D.TRAINING, [U(1, 4, 8), U(1, 4, 12)], [U(1, 4, 8), U(1, 4, 12), U(1, 4, 24), U(1, 4, 28)])
    same_as_oracle([actor2, critic2])
    same_as_oracle([D.StageChange(D.INFERENCE, [U(2, 1, 0)], [U(2, 1, 8)])])
    a = D.StageChange(D.GENERATION, [U(1, 1, 0)], [U(1, 1, 0), U(1, 1, 1)])
    b = D.StageChange(D.TRAINING, [U(1, 1, 1)], [U(1, 1, 1)])
    assert same_as_oracle([a, b], 1 << 20) is None                      # infeasible on both sides


def test_library_planner_on_random_plan_changes():
    """Random pools of 32-64 GPUs, 2-5 model-stages, power-of-two layouts, random placements and capacities:
    the two planners agree on every unit, primitive, edge and on the schedule, or both say infeasible."""
    rng = random.Random(7)
    agree = infeasible = 0
    for trial in range(300):
        n_gpus = rng.choice([32, 48, 64])
        changes = []
        for m in range(rng.randint(2, 5)):
            def collection():
                tp, pp = rng.choice([1, 2, 4, 8]), rng.choice([1, 2, 4])
                dp = rng.randint(1, 3)
                units = []
                for _ in range(dp):
                    first = rng.randrange(0, n_gpus - tp * pp + 1, tp * pp)
                    units.append(D.Unit(tp, pp, tuple(range(first, first + tp * pp))))
                return units
            changes.append(D.StageChange(rng.choice([0, 1, 2]), collection(), collection(),
                                         rng.choice([8, 16, 70]) << 20))
        cap = rng.choice([0, 64 << 20, 24 << 20, 12 << 20])
        if same_as_oracle(changes, cap) is None:
            infeasible += 1
        else:
            agree += 1
    assert agree > 100 and infeasible > 10


# ---------------------------------------------------------------- lowering the DAG to one task table

import numpy as np  # noqa: E402

from oracle import oracle as O  # noqa: E402
from paper_2609_34645_b200 import inputs as I  # noqa: E402
from test_compiler_cpu import desc_of, interpret, omodel_of, payload_mask, random_src  # noqa: E402


def lowered(changes, shapes, capacity=0):
    dag = B.Dag()
    for ch in changes:
        s = dag.add_stage(ch.kind, ch.state_bytes)
        for u in ch.current:
            dag.add_unit(s, False, u.tp, u.pp, list(u.gpus))
        for u in ch.target:
            dag.add_unit(s, True, u.tp, u.pp, list(u.gpus))
    dag.plan(capacity)
    descs = [desc_of(sh) for sh in shapes]
    return dag, dag.lower(descs), descs


def test_lowered_paper_example_equals_the_direct_reshard():
    """(TP4, PP8) -> four (TP4, PP2) replicas -> (TP8, PP2), executed from the lowered table level by level:
    the replicas equal the oracle's (TP4,PP8)->(TP4,PP2), the target equals its direct (TP4,PP8)->(TP8,PP2)."""
    sh = I.MICRO
    ch = D.StageChange(D.INFERENCE, [U(4, 8, 0)], [U(8, 2, 0)])
    dag, t, descs = lowered([ch], [sh])
    units, prims = dag.units(), dag.prims()
    assert [p["op"] for p in prims] == [B.OP_SPLIT, B.OP_DESTROY, B.OP_DESTROY, B.OP_MERGE]
    n_src, n_dst = t.num_buffers()
    assert n_src == 32 and n_dst == 4 * 8 + 16
    assert t.num_tiles()[1] == 2                                  # Split, then Merge
    m = omodel_of(sh)
    src = random_src(m, O.Plan(4, 8), 3, "bf16")
    got = [np.full(t.buffer_bytes(True, j), 0xA5, np.uint8) for j in range(n_dst)]
    interpret(t.rects(), src, got)
    sub_want = O.reshard(m, O.Plan(4, 8), O.Plan(4, 2), src, fill=0xA5)
    for k in range(4):
        for g, w in zip(got[8 * k:8 * k + 8], sub_want):
            assert np.array_equal(g, w)
    for g, w in zip(got[32:], O.reshard(m, O.Plan(4, 8), O.Plan(8, 2), src, fill=0xA5)):
        assert np.array_equal(g, w)
    # target shard i is cut from the sub-unit that sits on its GPU: shards 0..7 from replica 0, 8..15 from 1
    merge = [r for r in t.rects() if r.level == 1]
    assert {(r.dst_buf - n_src - 32) // 8 for r in merge} == {0, 1}
    assert all((r.src_buf - n_src) // 8 == (r.dst_buf - n_src - 32) // 8 for r in merge)
    rd, wr = t.bytes()
    one = descs[0].compile(B.Plan(4, 8), B.Plan(4, 2)).bytes()
    assert rd == one[0] + descs[0].compile(B.Plan(4, 2), B.Plan(8, 2)).bytes()[0] and wr > 4 * one[1]


def test_lowered_extend_then_merge():
    """Section 5.1's actor: (TP1, PP4) x2 -> (TP2, PP4) x2 = two Extends and two Merges; both target units hold
    the same logical state as the two source replicas."""
    sh = I.MICRO
    actor = D.StageChange(D.GENERATION, [U(1, 4, 0), U(1, 4, 4)],
                          [D.Unit(2, 4, tuple(range(0, 4)) + tuple(range(16, 20))),
                           D.Unit(2, 4, tuple(range(4, 8)) + tuple(range(20, 24)))])
    dag, t, descs = lowered([actor], [sh])
    m = omodel_of(sh)
    one = random_src(m, O.Plan(1, 4), 5, "bf16")
    src = one + [x.copy() for x in one]                          # DP replicas hold the same logical state
    n_src, n_dst = t.num_buffers()
    assert (n_src, n_dst) == (8, 2 * 4 + 2 * 8)
    got = [np.full(t.buffer_bytes(True, j), 0xA5, np.uint8) for j in range(n_dst)]
    interpret(t.rects(), src, got)
    want = O.reshard(m, O.Plan(1, 4), O.Plan(2, 4), one, fill=0xA5)
    for k in range(2):
        for g, w in zip(got[8 + 8 * k:16 + 8 * k], want):
            assert np.array_equal(g, w)


def test_lowered_random_dags_reach_the_target_state():
    """Random plan changes of one or two model-stages on the MICRO shape: whatever mix of Split, Extend, Merge
    and resource edges the planner produces, executing the lowered table level by level leaves every target
    unit equal to the direct reshard of the stage's logical state into the target layout."""
    sh = I.MICRO
    m = omodel_of(sh)
    rng = random.Random(11)
    ran = 0
    for trial in range(40):
        changes, logical = [], []
        for s in range(rng.randint(1, 2)):
            def collection():
                tp, pp = rng.choice([1, 2, 4, 8]), rng.choice([1, 2, 4])
                units = []
                for _ in range(rng.randint(1, 2)):
                    first = rng.randrange(0, 64 - tp * pp + 1, tp * pp)
                    units.append(D.Unit(tp, pp, tuple(range(first, first + tp * pp))))
                return units
            changes.append(D.StageChange(rng.choice([0, 1, 2]), collection(), collection(), 8 << 20))
            logical.append(random_src(m, O.Plan(1, 1), 100 * trial + s, "bf16"))
        try:
            dag, t, descs = lowered(changes, [sh] * len(changes))
        except B.NereusError as e:
            assert e.code in (B.ERR_UNSUPPORTED, B.ERR_INFEASIBLE)
            continue
        units, prims = dag.units(), dag.prims()
        created = {u for p in prims for u in p["dst"]}
        src, dst_units = [], []
        for u, (stage, tp, pp, gpus) in enumerate(units):
            if u not in created:                       # DP replicas of a stage hold the same logical state
                src += O.reshard(m, O.Plan(1, 1), O.Plan(tp, pp), logical[stage], fill=0xA5)
            else:
                dst_units.append(u)
        n_src, n_dst = t.num_buffers()
        assert n_src == len(src)
        got = [np.full(t.buffer_bytes(True, j), 0xA5, np.uint8) for j in range(n_dst)]
        interpret(t.rects(), src, got)
        at = 0
        for u in dst_units:
            stage, tp, pp, gpus = units[u]
            want = O.reshard(m, O.Plan(1, 1), O.Plan(tp, pp), logical[stage], fill=0xA5)
            for g, w in zip(got[at:at + tp * pp], want):
                assert np.array_equal(g, w), (trial, u)
            at += tp * pp
        ran += 1
    assert ran >= 15
