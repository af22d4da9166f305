"""TEST INFRASTRUCTURE -- NOT PART OF THE PRODUCT.

What Section 6.1 ("Decomposition and DAG Construction") and Section 6.2 ("DAG Execution and Safety") fix about
a transition DAG over EMU primitives, written as CHECKS of a finished plan rather than as a second planner.
`violations()` takes the plan changes and what a planner answered (units, primitives, state edges, resource
edges, serial order, levels) and returns every rule the answer breaks; `serial_orders_exist()` decides
feasibility of a handful of primitives by exhaustive search.  Nothing here builds a DAG, picks a Destroy or
sorts a ready set, so it cannot agree with a planner by construction.

Rules checked, each with the passage it restates:

  R1  T_sub is the largest layout both the current and the target units split into; the worked example
      (TP4, PP8) -> (TP8, PP2) goes through (TP4, PP2), hence (gcd tp, gcd pp).                  [6.1, par. 2]
  R2  Split(EMU, T_sub) turns one unit into k = tp*pp / |T_sub| independent units of layout T_sub on the
      same GPU set.                                                                             [5.2 (a)]
  R3  Merge fuses k replicas of one model-stage (layout T_sub) into one unit of the target layout T*.
                                                                                                 [5.2 (b)]
  R4  Extend replicates a unit onto a disjoint GPU set, same model-stage, same layout.           [5.2 (c)]
  R5  Destroy terminates a redundant unit: another replica of the model-stage retains the state;
      a transition that stops partway loses no logical state.                            [5.2 (d), 6.2 safety]
  R6  The local DAG runs Split -> Destroy -> Extend -> Merge, except that a unit an Extend copies is
      destroyed only after that Extend (and, source buffers staying live until their readers complete, is
      not merged away before it either).                                            [6.1, par. 2; 6.2 safety]
  R7  Every primitive waits for the primitives that produce the units it reads.                 [6.2, par. 1]
  R8  After the transition each model-stage holds exactly its target collection.                [6.1, par. 1]
  R9  State and resource edges together are acyclic; the serial order and the levels respect them.
                                                                                                 [6.1, par. 3]
  R10 A resource-dependency edge ends at a primitive that releases memory on a GPU its dependent acquires,
      and that primitive does not depend on the dependent.                                      [6.1, par. 3]
  R11 Release-before-acquire, then stage order generation -> inference -> training: when the serial order
      takes an acquisition, no Destroy was ready, and every ready acquisition of an earlier stage kind that
      it overtook did not fit at that moment.                                                   [6.1, par. 3]
  R12 The per-GPU capacity bound holds at every operation: in the serial order, with all primitives of one
      level running together, and in any execution that starts a primitive when its predecessors are done
      and its memory is free; such an execution never comes to a circular wait.        [6.2 safety, 6.1 par. 3]

The resource model is the one the product's header states (the paper gives the rules, not the bookkeeping):
a unit of layout (tp, pp) keeps state_bytes // (tp*pp) on each of its GPUs; Split, Extend and Merge need room
for what they create before they start; Split, Destroy and Merge free what they consume when they complete.
"""
from __future__ import annotations

import math
import random
from dataclasses import dataclass

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
    kind: int                    # GENERATION, INFERENCE or TRAINING
    current: list                # units of the current collection E_M
    target: list                 # units of the target collection E*_M
    state_bytes: int = 1 << 20   # bytes of one replica's state (theta, omega)


def t_sub(cur: Unit, tgt: Unit):
    """R1."""
    return math.gcd(cur.tp, tgt.tp), math.gcd(cur.pp, tgt.pp)


class _Memory:
    """Bytes resident per GPU while primitives start and finish."""

    def __init__(self, changes, units, live):
        self.changes, self.units = changes, units
        self.used = {}
        for u in live:
            self._add(u, +1)

    def shard(self, u):
        stage, tp, pp, _ = self.units[u]
        return self.changes[stage].state_bytes // (tp * pp)

    def _add(self, u, sign):
        for g in self.units[u][3]:
            self.used[g] = self.used.get(g, 0) + sign * self.shard(u)

    def need(self, p):
        n = {}
        if p["op"] in (SPLIT, EXTEND, MERGE):
            for d in p["dst"]:
                for g in self.units[d][3]:
                    n[g] = n.get(g, 0) + self.shard(d)
        return n

    def fits(self, p, capacity):
        return all(self.used.get(g, 0) + b <= capacity for g, b in self.need(p).items())

    def start(self, p):
        for d in p["dst"]:
            self._add(d, +1)

    def finish(self, p):
        if p["op"] in (SPLIT, DESTROY, MERGE):
            for s in p["src"]:
                self._add(s, -1)

    def freed_gpus(self, p):
        return {g for s in p["src"] for g in self.units[s][3]} if p["op"] in (SPLIT, DESTROY, MERGE) else set()


def _reach(prims):
    """ancestors[i] = every primitive i depends on, directly or transitively (None on a cycle)."""
    n = len(prims)
    anc, state = [set() for _ in range(n)], [0] * n

    def visit(i):
        if state[i] == 1:
            return False
        if state[i] == 2:
            return True
        state[i] = 1
        for d in prims[i]["deps"] | prims[i]["resource_deps"]:
            if not visit(d):
                return False
            anc[i] |= anc[d] | {d}
        state[i] = 2
        return True

    for i in range(n):
        if not visit(i):
            return None
    return anc


def violations(changes, capacity, units, prims, executions=20, seed=0):
    """Every rule of the module docstring that the plan (units, prims) breaks, as a list of strings.
    units: [(stage, tp, pp, gpus)], the current units first in input order; prims: [{op, stage, src, dst, deps,
    resource_deps, order, level}].  capacity 0 = unlimited."""
    bad = []
    cap = capacity or (1 << 62)
    n_cur = sum(len(ch.current) for ch in changes)
    flat = [(m, u) for m, ch in enumerate(changes) for u in ch.current]
    for i, (m, u) in enumerate(flat):
        if i >= len(units) or units[i] != (m, u.tp, u.pp, tuple(u.gpus)):
            bad.append(f"unit {i} is not current unit {u} of stage {m}")
    if bad:
        return bad
    producer, consumers = {}, {}
    for i, p in enumerate(prims):
        for d in p["dst"]:
            if d in producer or d < n_cur:
                bad.append(f"unit {d} is created twice or was there from the start")
            producer[d] = i
        for s in p["src"]:
            consumers.setdefault(s, []).append(i)

    # ---- per primitive: R1-R4, R7
    for i, p in enumerate(prims):
        m, op = p["stage"], p["op"]
        ch = changes[m]
        ts = t_sub(ch.current[0], ch.target[0])
        size = ts[0] * ts[1]
        lay = lambda u: units[u][1:3]
        if any(units[u][0] != m for u in p["src"] + p["dst"]):
            bad.append(f"prim {i} touches a unit of another model-stage")
        for s in p["src"]:
            if s in producer and producer[s] not in p["deps"]:
                bad.append(f"R7: prim {i} does not wait for prim {producer[s]}, which creates unit {s}")
        if op == SPLIT:
            cur = (ch.current[0].tp, ch.current[0].pp)
            if len(p["src"]) != 1 or lay(p["src"][0]) != cur or cur == ts:
                bad.append(f"R2: split {i} does not take one unit of the current layout {cur} != T_sub {ts}")
                continue
            k = cur[0] * cur[1] // size
            if len(p["dst"]) != k or any(lay(d) != ts for d in p["dst"]):
                bad.append(f"R1/R2: split {i} does not make {k} units of T_sub {ts}")
            got = [g for d in p["dst"] for g in units[d][3]]
            if sorted(got) != sorted(units[p["src"][0]][3]):
                bad.append(f"R2: split {i} leaves the unit's GPU set")
            if p["deps"]:
                bad.append(f"R6: split {i} waits for something")
        elif op == DESTROY:
            if len(p["src"]) != 1 or p["dst"]:
                bad.append(f"R5: destroy {i} must take one unit and make none")
        elif op == EXTEND:
            if len(p["src"]) != 1 or len(p["dst"]) != 1 or lay(p["src"][0]) != ts or lay(p["dst"][0]) != ts:
                bad.append(f"R4/R6: extend {i} does not copy one T_sub unit into one T_sub unit")
                continue
            if set(units[p["src"][0]][3]) & set(units[p["dst"][0]][3]):
                bad.append(f"R4: extend {i} writes onto its source's GPUs")
            if any(prims[d]["op"] != SPLIT for d in p["deps"]):
                bad.append(f"R6: extend {i} waits for something other than a split")
        elif op == MERGE:
            tgt = (ch.target[0].tp, ch.target[0].pp)
            k = tgt[0] * tgt[1] // size
            if tgt == ts or len(p["src"]) != k or any(lay(s) != ts for s in p["src"]) or len(p["dst"]) != 1 \
                    or lay(p["dst"][0]) != tgt:
                bad.append(f"R3: merge {i} does not fuse {k} units of T_sub {ts} into one of {tgt}")
                continue
            if [g for s in p["src"] for g in units[s][3]] != list(units[p["dst"][0]][3]):
                bad.append(f"R3: merge {i}: the target's GPUs are not its sub-units' GPUs, slot by slot")
            if any(prims[d]["op"] not in (SPLIT, EXTEND) for d in p["deps"]):
                bad.append(f"R6: merge {i} waits for a destroy or a merge")
    # R6: a unit that an Extend copies is given up (destroyed, or merged away) only after that Extend; apart
    # from those readers a Destroy waits for its unit's split at most
    for i, p in enumerate(prims):
        if p["op"] not in (DESTROY, MERGE):
            continue
        readers = {j for u in p["src"] for j in consumers.get(u, []) if prims[j]["op"] == EXTEND}
        if not readers <= p["deps"]:
            bad.append(f"R6: {OP_NAMES[p['op']]} {i} does not wait for the extends {sorted(readers - p['deps'])} "
                       "that copy a unit it gives up")
        for d in p["deps"] - readers:
            if p["op"] == DESTROY and prims[d]["op"] != SPLIT:
                bad.append(f"R6: destroy {i} waits for prim {d}, which is neither its unit's split nor a reader")
    # a unit is consumed (split, destroyed or merged away) at most once
    for u, cs in consumers.items():
        if sum(prims[j]["op"] != EXTEND for j in cs) > 1:
            bad.append(f"unit {u} is consumed twice")

    # ---- R9: one acyclic graph, an order and levels that respect it
    anc = _reach(prims)
    if anc is None:
        return bad + ["R9: state and resource edges form a cycle"]
    order = sorted(range(len(prims)), key=lambda i: prims[i]["order"])
    if sorted(p["order"] for p in prims) != list(range(len(prims))):
        return bad + ["R9: the serial order is not a permutation"]
    for i, p in enumerate(prims):
        preds = p["deps"] | p["resource_deps"]
        if any(prims[d]["order"] >= p["order"] for d in preds):
            bad.append(f"R9: prim {i} is scheduled before a predecessor")
        want = 1 + max((prims[d]["level"] for d in preds), default=-1)
        if p["level"] != want:
            bad.append(f"R9: prim {i} has level {p['level']}, its longest path says {want}")

    # ---- R10
    mem0 = _Memory(changes, units, range(n_cur))
    for i, p in enumerate(prims):
        for r in p["resource_deps"]:
            if not (mem0.freed_gpus(prims[r]) & set(mem0.need(p))):
                bad.append(f"R10: resource edge {r} -> {i}: prim {r} frees nothing on a GPU prim {i} acquires")
            if i in anc[r]:
                bad.append(f"R10: resource edge {r} -> {i}: prim {r} depends on prim {i}")

    # ---- serial replay: R5, R8, R11, R12
    mem = _Memory(changes, units, range(n_cur))
    live = {m: set() for m in range(len(changes))}
    for u in range(n_cur):
        live[units[u][0]].add(u)
    done = set()
    for step, i in enumerate(order):
        p = prims[i]
        ready = [j for j, q in enumerate(prims) if j not in done and (q["deps"] | q["resource_deps"]) <= done]
        if p["op"] != DESTROY:
            if any(prims[j]["op"] == DESTROY for j in ready):
                bad.append(f"R11: step {step} takes acquisition {i} while a destroy is ready")
            for j in ready:
                q = prims[j]
                if q["op"] != DESTROY and changes[q["stage"]].kind < changes[p["stage"]].kind and mem.fits(q, cap):
                    bad.append(f"R11: step {step} takes prim {i} before prim {j} of an earlier stage kind that fits")
        if not all(s in live[p["stage"]] for s in p["src"]):
            bad.append(f"prim {i} reads a unit that is not live at step {step}")
        if not mem.fits(p, cap):
            bad.append(f"R12: prim {i} does not fit at step {step} of the serial order")
        mem.start(p)
        mem.finish(p)
        live[p["stage"]] |= set(p["dst"])
        if p["op"] != EXTEND:
            live[p["stage"]] -= set(p["src"])
        if not live[p["stage"]]:
            bad.append(f"R5: after prim {i} model-stage {p['stage']} holds no copy of its state")
        done.add(i)
    for m, ch in enumerate(changes):
        got = sorted(units[u][1:] for u in live[m])
        want = sorted((u.tp, u.pp, tuple(u.gpus)) for u in ch.target)
        if got != want:
            bad.append(f"R8: model-stage {m} ends with {got}, its target collection is {want}")

    # ---- R12: all primitives of one level together
    mem = _Memory(changes, units, range(n_cur))
    for lvl in sorted({p["level"] for p in prims}):
        group = [p for p in prims if p["level"] == lvl]
        need = {}
        for p in group:
            for g, b in mem.need(p).items():
                need[g] = need.get(g, 0) + b
        over = [g for g, b in need.items() if mem.used.get(g, 0) + b > cap]
        if over:
            bad.append(f"R12: level {lvl} run together exceeds the capacity on GPUs {sorted(over)[:4]}")
        for p in group:
            mem.start(p)
        for p in group:
            mem.finish(p)

    # ---- R12: random executions under the readiness rule never exceed the bound and never get stuck
    rng = random.Random(seed)
    for _ in range(executions):
        mem = _Memory(changes, units, range(n_cur))
        running, finished = [], set()
        while len(finished) < len(prims):
            startable = [j for j, q in enumerate(prims)
                         if j not in finished and j not in running
                         and (q["deps"] | q["resource_deps"]) <= finished and mem.fits(q, cap)]
            moves = [("start", j) for j in startable] + [("finish", j) for j in running]
            if not moves:
                bad.append("R12: an execution came to a circular wait: "
                           f"{len(finished)} of {len(prims)} primitives done, nothing can start")
                break
            what, j = rng.choice(moves)
            if what == "start":
                mem.start(prims[j])
                running.append(j)
            else:
                mem.finish(prims[j])
                running.remove(j)
                finished.add(j)
            if any(v > cap for v in mem.used.values()):
                bad.append("R12: an execution exceeded the capacity bound")
                break
    return bad


def serial_orders_exist(changes, capacity, units, prims, limit=10, paper_rules=False):
    """Exhaustive search: is there ANY serial order of the primitives that respects the state edges (resource
    edges are the planner's own additions and are ignored) and the capacity bound at every step?  With
    paper_rules the order must also obey the two combination rules of Section 6.1 (R11): a ready Destroy goes
    before any acquisition, and among the ready acquisitions that fit only one of the earliest stage kind may
    be taken (every such one is tried: the paper names no further tie-break).  For small cases only (at most
    `limit` primitives); returns None beyond that."""
    if len(prims) > limit:
        return None
    cap = capacity or (1 << 62)
    n_cur = sum(len(ch.current) for ch in changes)
    seen = set()

    def search(done):
        if len(done) == len(prims):
            return True
        if done in seen:
            return False
        seen.add(done)
        mem = _Memory(changes, units, range(n_cur))
        for j in sorted(done):                    # usage after a set of completed primitives is order-free
            mem.start(prims[j])
            mem.finish(prims[j])
        moves = [j for j, q in enumerate(prims) if j not in done and q["deps"] <= done and mem.fits(q, cap)]
        if paper_rules and moves:
            destroys = [j for j in moves if prims[j]["op"] == DESTROY]
            first = min(changes[prims[j]["stage"]].kind for j in moves)
            moves = destroys or [j for j in moves if changes[prims[j]["stage"]].kind == first]
        return any(search(done | {j}) for j in moves)

    return search(frozenset())
