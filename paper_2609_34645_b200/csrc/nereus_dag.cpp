// Transition DAG over EMU primitives: local DAGs per model-stage in the order Split -> Destroy -> Extend ->
// Merge through T_sub, then one global schedule with resource-dependency edges (Section 6.1 of the Nereus
// paper).  Host only.
#include <algorithm>
#include <map>
#include <new>
#include <numeric>
#include <set>
#include <vector>

#include "nereus_internal.hpp"

using namespace nereus;

namespace {

struct Planner {
    nereus_dag_s&                               g;
    uint64_t                                    capacity;
    std::map<int, int>                          producer;    // unit -> primitive that creates it
    std::map<int, uint64_t>                     used;        // gpu -> resident bytes
    std::map<int, std::vector<std::pair<int, uint64_t>>> released;   // gpu -> (primitive, bytes freed), in order

    int add_unit(int stage, int tp, int pp, std::vector<int> gpus) {
        g.units.push_back(UnitRec{stage, tp, pp, std::move(gpus)});
        return (int)g.units.size() - 1;
    }
    int add_prim(int op, int stage, std::vector<int> src, std::vector<int> dst) {
        PrimRec p;
        p.op = op; p.stage = stage; p.src = std::move(src); p.dst = std::move(dst);
        for (int u : p.src) {
            auto it = producer.find(u);
            if (it != producer.end()) p.deps.insert(it->second);
        }
        g.prims.push_back(p);
        const int id = (int)g.prims.size() - 1;
        for (int u : g.prims[id].dst) producer[u] = id;
        return id;
    }
    uint64_t shard_bytes(int u) const {
        const UnitRec& x = g.units[u];
        return g.stages[x.stage].state_bytes / (uint64_t)(x.tp * x.pp);
    }
    void occupy(int u, bool add) {
        for (int gpu : g.units[u].gpus) {
            if (add) used[gpu] += shard_bytes(u);
            else     used[gpu] -= shard_bytes(u);
        }
    }

    // ---- one model-stage: Split, then Destroy, then Extend, then Merge
    int local_dag(int m, const std::vector<int>& current_ids) {
        const StageRec& st = g.stages[m];
        const int tps = std::gcd(st.current[0].tp, st.target[0].tp);
        const int pps = std::gcd(st.current[0].pp, st.target[0].pp);
        const int s = tps * pps;
        std::vector<int> subs;
        for (size_t i = 0; i < st.current.size(); ++i) {
            const UnitRec& u = st.current[i];
            if (u.tp == tps && u.pp == pps) { subs.push_back(current_ids[i]); continue; }
            const int k = u.tp * u.pp / s;
            std::vector<int> made;
            for (int j = 0; j < k; ++j)
                made.push_back(add_unit(m, tps, pps, std::vector<int>(u.gpus.begin() + j * s, u.gpus.begin() + (j + 1) * s)));
            add_prim(NEREUS_OP_SPLIT, m, {current_ids[i]}, made);
            subs.insert(subs.end(), made.begin(), made.end());
        }
        // the target's slots
        struct Slot { int target; std::vector<int> gpus; int unit; };
        std::vector<Slot> slots;
        for (size_t t = 0; t < st.target.size(); ++t) {
            const UnitRec& v = st.target[t];
            for (int j = 0; j < v.tp * v.pp / s; ++j)
                slots.push_back(Slot{(int)t, std::vector<int>(v.gpus.begin() + j * s, v.gpus.begin() + (j + 1) * s), -1});
        }
        std::map<std::vector<int>, int> at;              // GPU group -> sub-unit sitting there (last one wins)
        for (int u : subs) at[g.units[u].gpus] = u;
        std::set<int> kept;
        for (Slot& sl : slots) {
            auto it = at.find(sl.gpus);
            if (it != at.end() && !kept.count(it->second)) { kept.insert(it->second); sl.unit = it->second; }
        }
        std::map<int, int> destroy_of;
        std::map<int, std::vector<int>> readers;          // unit -> Extends that copy it
        for (int u : subs)
            if (!kept.count(u)) destroy_of[u] = add_prim(NEREUS_OP_DESTROY, m, {u}, {});
        // Extend copies onto a GPU set disjoint from its source's (Section 5.2(c)): per empty slot, the
        // lowest-numbered kept sub-unit that shares no GPU with the slot, else the lowest-numbered such sub-unit
        // at all; a slot that overlaps every sub-unit without coinciding with one cannot be filled by the
        // paper's primitives
        auto disjoint = [this](int u, const std::vector<int>& gpus) {
            for (int a : g.units[u].gpus)
                if (std::find(gpus.begin(), gpus.end(), a) != gpus.end()) return false;
            return true;
        };
        for (Slot& sl : slots) {
            if (sl.unit >= 0) continue;
            int source = -1;
            for (int u : kept)
                if (disjoint(u, sl.gpus)) { source = u; break; }
            if (source < 0) {
                std::vector<int> sorted_subs(subs);
                std::sort(sorted_subs.begin(), sorted_subs.end());
                for (int u : sorted_subs)
                    if (disjoint(u, sl.gpus)) { source = u; break; }
            }
            if (source < 0) return NEREUS_ERR_UNSUPPORTED;
            sl.unit = add_unit(m, tps, pps, sl.gpus);
            const int e = add_prim(NEREUS_OP_EXTEND, m, {source}, {sl.unit});
            readers[source].push_back(e);
            auto it = destroy_of.find(source);
            if (it != destroy_of.end()) g.prims[it->second].deps.insert(e);     // the last copy goes after the Extend
        }
        for (size_t t = 0; t < st.target.size(); ++t) {
            const UnitRec& v = st.target[t];
            if (v.tp == tps && v.pp == pps) continue;
            std::vector<int> mine;
            for (const Slot& sl : slots)
                if (sl.target == (int)t) mine.push_back(sl.unit);
            const int tu = add_unit(m, v.tp, v.pp, v.gpus);
            const int mg = add_prim(NEREUS_OP_MERGE, m, mine, {tu});
            // a Merge frees the sub-units it fuses: like a Destroy it waits for the Extends that still copy them
            for (int u : mine)
                for (int e : readers[u]) g.prims[mg].deps.insert(e);
        }
        return NEREUS_OK;
    }

    std::set<int> ancestors(int pid) const {
        std::set<int> seen;
        std::vector<int> todo{pid};
        while (!todo.empty()) {
            const int x = todo.back(); todo.pop_back();
            for (const std::set<int>* e : {&g.prims[x].deps, &g.prims[x].rdeps})
                for (int d : *e)
                    if (seen.insert(d).second) todo.push_back(d);
        }
        return seen;
    }
    std::map<int, uint64_t> needs(const PrimRec& p) const {
        std::map<int, uint64_t> need;
        if (p.op != NEREUS_OP_DESTROY)
            for (int d : p.dst)
                for (int gpu : g.units[d].gpus) need[gpu] += shard_bytes(d);
        return need;
    }
    void apply(int pid) {
        PrimRec& p = g.prims[pid];
        for (int d : p.dst) occupy(d, true);
        if (p.op != NEREUS_OP_EXTEND)
            for (int u : p.src) {
                occupy(u, false);
                for (int gpu : g.units[u].gpus) released[gpu].push_back({pid, shard_bytes(u)});
            }
    }
    bool before(int a, int b) const {                      // schedule priority
        const PrimRec& x = g.prims[a]; const PrimRec& y = g.prims[b];
        const int xa[4] = {x.op == NEREUS_OP_DESTROY ? 0 : 1, g.stages[x.stage].kind, x.stage, a};
        const int ya[4] = {y.op == NEREUS_OP_DESTROY ? 0 : 1, g.stages[y.stage].kind, y.stage, b};
        return std::lexicographical_compare(xa, xa + 4, ya, ya + 4);
    }
    bool satisfied(const PrimRec& p, const std::vector<char>& done) const {
        for (int d : p.deps) if (!done[d]) return false;
        for (int d : p.rdeps) if (!done[d]) return false;
        return true;
    }

    int schedule() {
        const int n = (int)g.prims.size();
        std::vector<char> done(n, 0);
        int n_done = 0;
        while (n_done < n) {
            std::vector<int> ready;
            for (int i = 0; i < n; ++i)
                if (!done[i] && satisfied(g.prims[i], done)) ready.push_back(i);
            if (ready.empty()) return NEREUS_ERR_INFEASIBLE;
            std::sort(ready.begin(), ready.end(), [this](int a, int b) { return before(a, b); });
            bool progressed = false;
            for (int pid : ready) {
                PrimRec& p = g.prims[pid];
                const std::set<int> anc = ancestors(pid);
                std::vector<int> rely, short_gpus;
                for (const auto& [gpu, need] : needs(p)) {
                    // memory freed by primitives p does not depend on cannot be counted on
                    std::vector<std::pair<int, uint64_t>> extra;
                    auto it = released.find(gpu);
                    if (it != released.end())
                        for (const auto& rel : it->second)
                            if (!anc.count(rel.first) && std::find(rely.begin(), rely.end(), rel.first) == rely.end())
                                extra.push_back(rel);
                    uint64_t level = used[gpu];
                    for (const auto& rel : extra) level += rel.second;
                    for (auto r = extra.rbegin(); r != extra.rend(); ++r) {   // newest release first
                        if (level + need <= capacity) break;
                        rely.push_back(r->first);
                        level -= r->second;
                    }
                    if (level + need > capacity) short_gpus.push_back(gpu);
                }
                if (short_gpus.empty()) {
                    p.rdeps.insert(rely.begin(), rely.end());
                    apply(pid);
                    done[pid] = 1; ++n_done;
                    p.order = n_done - 1;
                    progressed = true;
                    break;
                }
                // blocked: an executable Destroy that frees one of the GPUs and does not depend on p
                int pick = -1;
                for (int i = 0; i < n; ++i) {
                    const PrimRec& q = g.prims[i];
                    if (q.op != NEREUS_OP_DESTROY || done[i] || !satisfied(q, done)) continue;
                    bool touches = false;
                    for (int gpu : g.units[q.src[0]].gpus)
                        if (std::find(short_gpus.begin(), short_gpus.end(), gpu) != short_gpus.end()) touches = true;
                    if (!touches || ancestors(i).count(pid)) continue;
                    if (pick < 0 || before(i, pick)) pick = i;
                }
                if (pick >= 0) {
                    p.rdeps.insert(pick);
                    progressed = true;
                    break;
                }
            }
            if (!progressed) return NEREUS_ERR_INFEASIBLE;
        }
        // levels: longest path over state and resource edges, in schedule order
        std::vector<int> by_order(n);
        for (int i = 0; i < n; ++i) by_order[g.prims[i].order] = i;
        for (int i : by_order) {
            int lv = 0;
            for (int d : g.prims[i].deps) lv = std::max(lv, g.prims[d].level + 1);
            for (int d : g.prims[i].rdeps) lv = std::max(lv, g.prims[d].level + 1);
            g.prims[i].level = lv;
        }
        return NEREUS_OK;
    }
};

}  // namespace

extern "C" {

int nereus_dag_create(nereus_dag_t* out) {
    if (!out) return NEREUS_ERR_ARG;
    try { *out = new nereus_dag_s(); } catch (const std::bad_alloc&) { return NEREUS_ERR_NOMEM; }
    return NEREUS_OK;
}

int nereus_dag_destroy(nereus_dag_t dag) {
    if (!dag) return NEREUS_ERR_ARG;
    delete dag;
    return NEREUS_OK;
}

int nereus_dag_add_stage(nereus_dag_t dag, int kind, uint64_t state_bytes, int* stage) {
    if (!dag || !stage || kind < NEREUS_GENERATION || kind > NEREUS_TRAINING || state_bytes == 0 || dag->planned)
        return NEREUS_ERR_ARG;
    try {
        dag->stages.push_back(StageRec{kind, state_bytes, {}, {}});
    } catch (const std::bad_alloc&) { return NEREUS_ERR_NOMEM; }
    *stage = (int)dag->stages.size() - 1;
    return NEREUS_OK;
}

int nereus_dag_add_unit(nereus_dag_t dag, int stage, int is_target, int tp, int pp, const int* gpus) {
    if (!dag || !gpus || stage < 0 || (size_t)stage >= dag->stages.size() || tp < 1 || pp < 1 || dag->planned)
        return NEREUS_ERR_ARG;
    try {
        UnitRec u{stage, tp, pp, std::vector<int>(gpus, gpus + tp * pp)};
        (is_target ? dag->stages[stage].target : dag->stages[stage].current).push_back(std::move(u));
    } catch (const std::bad_alloc&) { return NEREUS_ERR_NOMEM; }
    return NEREUS_OK;
}

int nereus_dag_plan(nereus_dag_t dag, uint64_t gpu_capacity) {
    if (!dag || dag->planned || dag->stages.empty()) return NEREUS_ERR_ARG;
    try {
        for (const StageRec& st : dag->stages) {
            if (st.current.empty() || st.target.empty()) return NEREUS_ERR_ARG;
            for (const UnitRec& u : st.current)
                if (u.tp != st.current[0].tp || u.pp != st.current[0].pp) return NEREUS_ERR_ARG;
            for (const UnitRec& u : st.target)
                if (u.tp != st.target[0].tp || u.pp != st.target[0].pp) return NEREUS_ERR_ARG;
        }
        Planner P{*dag, gpu_capacity ? gpu_capacity : ~0ull >> 2, {}, {}, {}};
        std::vector<std::vector<int>> current_ids(dag->stages.size());
        for (size_t m = 0; m < dag->stages.size(); ++m)
            for (const UnitRec& u : dag->stages[m].current)
                current_ids[m].push_back(P.add_unit((int)m, u.tp, u.pp, u.gpus));
        for (size_t m = 0; m < dag->stages.size(); ++m)
            if (int rc = P.local_dag((int)m, current_ids[m])) return rc;
        for (const auto& ids : current_ids)
            for (int u : ids) P.occupy(u, true);
        dag->planned = true;                       // frozen from here on: units and primitives exist
        const int rc = P.schedule();
        dag->scheduled = rc == NEREUS_OK;          // only a complete schedule may be lowered
        return rc;
    } catch (const std::bad_alloc&) { return NEREUS_ERR_NOMEM; }
}

int nereus_dag_num_units(nereus_dag_t dag, int* n) {
    if (!dag || !n) return NEREUS_ERR_ARG;
    *n = (int)dag->units.size();
    return NEREUS_OK;
}

int nereus_dag_unit(nereus_dag_t dag, int unit, int* stage, int* tp, int* pp, int* gpus, int gpus_cap) {
    if (!dag || unit < 0 || (size_t)unit >= dag->units.size() || !stage || !tp || !pp) return NEREUS_ERR_ARG;
    const UnitRec& u = dag->units[unit];
    *stage = u.stage; *tp = u.tp; *pp = u.pp;
    if (gpus) {
        if (gpus_cap < (int)u.gpus.size()) return NEREUS_ERR_ARG;
        std::copy(u.gpus.begin(), u.gpus.end(), gpus);
    }
    return NEREUS_OK;
}

int nereus_dag_num_prims(nereus_dag_t dag, int* n) {
    if (!dag || !n) return NEREUS_ERR_ARG;
    *n = (int)dag->prims.size();
    return NEREUS_OK;
}

int nereus_dag_prim(nereus_dag_t dag, int prim, nereus_prim_t* out) {
    if (!dag || !out || prim < 0 || (size_t)prim >= dag->prims.size()) return NEREUS_ERR_ARG;
    const PrimRec& p = dag->prims[prim];
    out->op = p.op; out->stage = p.stage;
    out->n_src = (int)p.src.size(); out->n_dst = (int)p.dst.size();
    out->n_deps = (int)p.deps.size(); out->n_resource_deps = (int)p.rdeps.size();
    out->order = p.order; out->level = p.level;
    return NEREUS_OK;
}

int nereus_dag_prim_lists(nereus_dag_t dag, int prim, int* src, int* dst, int* deps, int* resource_deps) {
    if (!dag || prim < 0 || (size_t)prim >= dag->prims.size()) return NEREUS_ERR_ARG;
    const PrimRec& p = dag->prims[prim];
    if (src) std::copy(p.src.begin(), p.src.end(), src);
    if (dst) std::copy(p.dst.begin(), p.dst.end(), dst);
    if (deps) std::copy(p.deps.begin(), p.deps.end(), deps);
    if (resource_deps) std::copy(p.rdeps.begin(), p.rdeps.end(), resource_deps);
    return NEREUS_OK;
}

}  // extern "C"
