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
