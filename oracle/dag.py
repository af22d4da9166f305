"""TEST INFRASTRUCTURE -- NOT PART OF THE PRODUCT.

Plain restatement of the transition-DAG construction of Section 6.1, step by step in the paper's order, for the
tests to hold the library's planner against.  It is a heuristic, so the oracle is the algorithm's steps, not
a closed form.

What the paper fixes (Section 6.1, with the primitives of Section 5.2):
  * per model-stage M the change Delta_M = (E_M -> E*_M) becomes a local DAG in the default order
    Split -> Destroy -> Extend -> Merge;
  * first the largest layout T_sub into which both the current and the target units can be split; the worked
    example (TP4, PP8) -> (TP8, PP2) goes through four (TP4, PP2) units, so T_sub = (gcd tp, gcd pp);
  * Split(EMU, T_sub) turns one unit into k replica units of layout T_sub on the same GPUs; Destroy removes
    redundant units and releases their GPUs; Extend adds replicas on the target GPUs; a unit with no other
    replica is destroyed only after Extend has copied it; Merge combines the intermediate units into the
    target layout and DP degree;
  * local DAGs are combined with two deterministic rules: release-before-acquire (resource-releasing
    primitives first) and stage order generation -> inference -> training; when an acquisition is blocked
    the engine selects an executable Destroy that releases the needed GPUs and inserts a resource-dependency
    edge; a Destroy that depends, directly or transitively, on the blocked acquisition is never selected; if
    no such Destroy exists the target plan fails the feasibility check.

What this build had to decide (readings, all repeated in the product's header):
  * sub-unit j of a split unit sits on the unit's GPUs [j*s, (j+1)*s), s = |T_sub|, in shard order;
  * a target unit's slots are its GPUs cut the same way; a slot already holding a sub-unit (same GPUs, same
    order) is kept in place, every other slot is filled by Extend from the lowest-numbered live sub-unit of
    the model-stage that is kept, else from the lowest-numbered one at all;
  * resources are bytes of GPU memory (the pool is assumed nearly full): a unit of layout (tp, pp) keeps
    state_bytes // (tp*pp) on each of its GPUs; every GPU has `gpu_capacity` bytes; Split needs room for the
    new sub-unit shards next to the old shard on each of the unit's GPUs and frees the old shard when it
    completes; Extend needs room for one shard on each target GPU; Merge needs room for the target shard
    next to the sub-unit shards and frees those when it completes;
  * ties among ready primitives: releasing before acquiring, then stage kind, then model-stage index, then
    primitive id.
"""
from __future__ import annotations

import math
from dataclasses import dataclass, field

GENERATION, INFERENCE, TRAINING = 0, 1, 2
SPLIT, DESTROY, EXTEND, MERGE = 0, 1, 2, 3
OP_NAMES = {SPLIT: "split", DESTROY: "destroy", EXTEND: "extend", MERGE: "merge"}


@dataclass(frozen=True)
class Unit:
    tp: int
    pp: int
    gpus: tuple


@dataclass
class StageChange:
    kind: int                 # GENERATION, INFERENCE or TRAINING
    current: list             # units of the current collection E_M
    target: list              # units of the target collection E*_M
    state_bytes: int = 1 << 20   # bytes of one replica's state (theta, omega)


@dataclass
class Prim:
    op: int
    stage: int
    src: tuple                # unit ids read
    dst: tuple                # unit ids created
    deps: set = field(default_factory=set)         # state dependencies (prim ids)
    resource_deps: set = field(default_factory=set)


class Infeasible(Exception):
    pass


def t_sub(cur: Unit, tgt: Unit):
    return math.gcd(cur.tp, tgt.tp), math.gcd(cur.pp, tgt.pp)


def plan(changes: list, gpu_capacity: int = 1 << 62):
    """Returns (units, prims, order): units = list of (stage, tp, pp, gpus) by unit id (current units first, in
    input order), prims = list of Prim, order = the serial schedule (prim ids)."""
    units, prims = [], []
    producer = {}                                   # unit id -> prim id that creates it

    def new_unit(stage, tp, pp, gpus):
        units.append((stage, tp, pp, tuple(gpus)))
        return len(units) - 1

    def new_prim(op, stage, src, dst):
        p = Prim(op, stage, tuple(src), tuple(dst))
        for u in src:
            if u in producer:
                p.deps.add(producer[u])
        prims.append(p)
        pid = len(prims) - 1
        for u in dst:
            producer[u] = pid
        return pid

    current_ids = []
    for m, ch in enumerate(changes):
        current_ids.append([new_unit(m, u.tp, u.pp, u.gpus) for u in ch.current])

    # ---- local DAGs, Split -> Destroy -> Extend -> Merge
    for m, ch in enumerate(changes):
        if not ch.current or not ch.target:
            raise ValueError("a model-stage needs at least one current and one target unit")
        tp_s, pp_s = t_sub(ch.current[0], ch.target[0])
        s = tp_s * pp_s
        # Split
        subs = []                                    # live sub-units (unit ids) of layout T_sub
        for uid, u in zip(current_ids[m], ch.current):
            if (u.tp, u.pp) == (tp_s, pp_s):
                subs.append(uid)
                continue
            k = u.tp * u.pp // s
            made = [new_unit(m, tp_s, pp_s, u.gpus[j * s:(j + 1) * s]) for j in range(k)]
            new_prim(SPLIT, m, [uid], made)
            subs += made
        # slots the target needs
        slots = []                                   # (target index, gpus)
        for ti, v in enumerate(ch.target):
            k_t = v.tp * v.pp // s
            for j in range(k_t):
                slots.append((ti, tuple(v.gpus[j * s:(j + 1) * s])))
        by_gpus = {units[u][3]: u for u in subs}
        kept, filled = set(), {}
        for si, (ti, g) in enumerate(slots):
            if g in by_gpus and by_gpus[g] not in kept:
                kept.add(by_gpus[g])
                filled[si] = by_gpus[g]
        redundant = [u for u in subs if u not in kept]
        # Extend sources: a kept sub-unit if there is one, else the lowest-numbered sub-unit
        source = min(kept) if kept else min(subs)
        pending_extends = []
        for si, (ti, g) in enumerate(slots):
            if si in filled:
                continue
            pending_extends.append((si, g))
        # Destroy (listed before Extend, but a unit that Extend still reads is destroyed after it)
        destroy_of = {}
        for u in redundant:
            destroy_of[u] = new_prim(DESTROY, m, [u], [])
        # Extend
        for si, g in pending_extends:
            nu = new_unit(m, tp_s, pp_s, g)
            pid = new_prim(EXTEND, m, [source], [nu])
            filled[si] = nu
            if source in destroy_of:
                prims[destroy_of[source]].deps.add(pid)
        # Merge
        for ti, v in enumerate(ch.target):
            mine = [filled[si] for si, (tj, g) in enumerate(slots) if tj == ti]
            if (v.tp, v.pp) == (tp_s, pp_s):
                continue                             # the slot's sub-unit is the target unit
            tu = new_unit(m, v.tp, v.pp, v.gpus)
            new_prim(MERGE, m, mine, [tu])

    # ---- global DAG: serial schedule under GPU slots, release-before-acquire, stage order
    used = {}                                        # gpu -> resident bytes

    def shard(u):                                    # bytes one GPU of unit u holds
        stage, tp, pp, _ = units[u]
        return changes[stage].state_bytes // (tp * pp)

    def occupy(u, sign=1):
        for g in units[u][3]:
            used[g] = used.get(g, 0) + sign * shard(u)

    for ids in current_ids:
        for u in ids:
            occupy(u)

    def needs(p):                                    # {gpu: bytes that must be free before p starts}
        need = {}
        if p.op in (SPLIT, EXTEND, MERGE):
            for d in p.dst:
                for g in units[d][3]:
                    need[g] = need.get(g, 0) + shard(d)
        return need

    released = {}                                    # gpu -> [(prim id, bytes it freed there)], in order

    def apply(pid):
        p = prims[pid]
        for d in p.dst:                              # new shards appear ...
            occupy(d)
        if p.op in (SPLIT, DESTROY, MERGE):          # ... and these primitives free what they consumed
            for sct in p.src:
                occupy(sct, -1)
                for g in units[sct][3]:
                    released.setdefault(g, []).append((pid, shard(sct)))

    def ancestors(pid):
        seen, todo = set(), [pid]
        while todo:
            x = todo.pop()
            for d in prims[x].deps | prims[x].resource_deps:
                if d not in seen:
                    seen.add(d)
                    todo.append(d)
        return seen

    def key(pid):
        p = prims[pid]
        return (0 if p.op == DESTROY else 1, changes[p.stage].kind, p.stage, pid)

    done, order = set(), []
    while len(done) < len(prims):
        ready = sorted((i for i, p in enumerate(prims)
                        if i not in done and (p.deps | p.resource_deps) <= done), key=key)
        if not ready:
            raise Infeasible("dependency cycle")
        progressed = False
        for pid in ready:
            p = prims[pid]
            anc = ancestors(pid)
            rely, short = [], []
            for g, n in sorted(needs(p).items()):
                # memory freed by primitives p does not depend on cannot be counted on: ready primitives run
                # concurrently, so p must wait for the releases it needs (a resource-dependency edge)
                extra = [(q, b) for q, b in released.get(g, []) if q not in anc and q not in rely]
                level = used.get(g, 0) + sum(b for _, b in extra)
                for q, b in reversed(extra):         # newest release first
                    if level + n <= gpu_capacity:
                        break
                    rely.append(q)
                    level -= b
                if level + n > gpu_capacity:
                    short.append(g)
            if not short:
                p.resource_deps |= set(rely)
                apply(pid)
                done.add(pid)
                order.append(pid)
                progressed = True
                break
            # blocked acquisition: an executable Destroy that releases one of the needed GPUs and does not
            # itself depend on the blocked primitive
            cands = [i for i, q in enumerate(prims)
                     if q.op == DESTROY and i not in done and set(units[q.src[0]][3]) & set(short)
                     and pid not in ancestors(i) and (q.deps | q.resource_deps) <= done]
            if cands:
                p.resource_deps.add(min(cands, key=key))
                progressed = True
                break                                 # the Destroy is ready and sorts first next round
        if not progressed:
            raise Infeasible("an acquisition is blocked and no executable Destroy releases its GPUs")
    return units, prims, order
