"""Pins of the CPU oracle against things other than itself (no GPU).

The paper prints no worked numeric example of a reshard; what it fixes is the semantic contract that Split and
Merge re-cut and move state without touching the logical state (Section 6.2), and one layout example,
(TP4, PP8) -> (TP4, PP2) units -> (TP8, PP2) (Section 6.1).  The pins are therefore: np.split /
np.concatenate special cases, a brute-force per-element owner function, identity, round trips, checksum
conservation, path independence through the paper's example, published parameter counts, and torch's
fp32 -> bf16 conversion over every fp32 bit pattern.
"""
import itertools
import os

import numpy as np
import pytest
import torch

import npmodel
from oracle import oracle as O
from paper_2609_34645_b200 import inputs as I

GOLDEN = os.path.join(os.path.dirname(__file__), "golden")


def model_of(sh, dtype=O.BF16, value_head=False):
    return O.Model(sh.layers, sh.hidden, sh.heads, sh.kv_heads, sh.ffn, sh.vocab, dtype, value_head)


def plans_for(sh, max_tp=8, max_pp=8):
    out = []
    for tp in (1, 2, 4, 8):
        for pp in (1, 2, 4, 8):
            if tp <= max_tp and pp <= max_pp and tp <= sh.kv_heads and sh.kv_heads % tp == 0 \
                    and sh.ffn % tp == 0 and sh.vocab % tp == 0 and sh.layers % pp == 0:
                out.append((tp, pp))
    return out


def payload_mask(model, plan):
    """Boolean mask per shard: True on bytes that belong to a tensor, False on padding."""
    masks = [np.zeros(O.shard_bytes(model, plan, s), bool) for s in range(O.num_shards(model, plan))]
    e = O.es(model, plan)
    for s in range(len(masks)):
        for t in range(O.num_logical(model)):
            p = O.locate(model, plan, s, t)
            if p.held:
                assert not masks[s][p.offset:p.offset + p.nr * p.nc * e].any(), "tensors overlap"
                masks[s][p.offset:p.offset + p.nr * p.nc * e] = True
    return masks


# ---------------------------------------------------------------- closed forms (published sizes)

@pytest.mark.parametrize("sh,vh,total", [
    (I.LLAMA_8B, False, 8_030_261_248),    # Llama-3-8B's published parameter count
    (I.LLAMA_8B, True, 7_504_928_768),     # LM head [128256, 4096] replaced by a [1, 4096] value head
    (I.DENSE_32B, False, 32_763_417_600),
    (I.TINY, False, 1_975_552),
])
def test_parameter_totals(sh, vh, total):
    m = model_of(sh, value_head=vh)
    assert O.num_logical(m) == 9 * sh.layers + 3
    assert sum(r * c for r, c in (O.logical_shape(m, t) for t in range(O.num_logical(m)))) == total


@pytest.mark.parametrize("sh,vh,total", [(I.LLAMA_8B, False, 8_030_261_248), (I.LLAMA_8B, True, 7_504_928_768),
                                         (I.TINY, False, 1_975_552)])
def test_shards_partition_the_model(sh, vh, total):
    """Under every plan the shards' parts tile each logical tensor exactly once (replicated tensors once per
    TP rank), and the parts fit in the shard without overlap."""
    m = model_of(sh, value_head=vh)
    for tp, pp in plans_for(sh, max_tp=4 if sh is I.LLAMA_8B else 8, max_pp=2 if sh is I.LLAMA_8B else 8):
        pl = O.Plan(tp, pp)
        n = O.num_shards(m, pl)
        assert n == tp * pp
        got = 0
        for t in range(O.num_logical(m)):
            rows, cols = O.logical_shape(m, t)
            parts = [O.locate(m, pl, s, t) for s in range(n)]
            held = [p for p in parts if p.held]
            area = sum(p.nr * p.nc for p in held)
            assert area in (rows * cols, tp * rows * cols)
            if area == tp * rows * cols and tp > 1:
                assert rows == 1          # only norms / value head are replicated
            got += rows * cols
            for s, p in enumerate(parts):
                if p.held:
                    assert p.offset % 256 == 0 or t != 0
                    assert p.offset + p.nr * p.nc * 2 <= O.shard_bytes(m, pl, s)
        assert got == total


def test_shard_sizes_8b_split():
    """8B bf16 TP4PP2: eight shards of about 2.008 GB, the two stages equal in size (embed vs head + ln_f)."""
    m = model_of(I.LLAMA_8B)
    sizes = [O.shard_bytes(m, O.Plan(4, 2), s) for s in range(8)]
    per_layer = (25_165_824 + 16_777_216 + 117_440_512 + 58_720_256) // 4 + 2 * 4096
    assert sizes[0] == (525_336_576 // 4 + 16 * per_layer) * 2
    assert sizes[4] == sizes[0] + 4096 * 2
    assert O.shard_bytes(m, O.Plan(1, 1), 0) == 8_030_261_248 * 2


# ---------------------------------------------------------------- np.split special cases

@pytest.mark.parametrize("sh", [I.TINY, I.MICRO])
@pytest.mark.parametrize("es", [2, 4])
@pytest.mark.parametrize("vh", [False, True])
def test_against_np_split(sh, es, vh):
    """TP1PP1 <-> any plan agrees with shards built by np.split / np.concatenate from numpy logical tensors
    (sentinel padding must survive: padding is never written)."""
    m = model_of(sh, O.BF16 if es == 2 else O.FP32, vh)
    logical = npmodel.random_logical(sh, es, seed=11, value_head=vh)
    full = npmodel.build_shards(sh, 1, 1, logical, vh)
    assert full[0].size == O.shard_bytes(m, O.Plan(1, 1), 0)
    for tp, pp in plans_for(sh):
        want = npmodel.build_shards(sh, tp, pp, logical, vh)
        got = O.reshard(m, O.Plan(1, 1), O.Plan(tp, pp), full, fill=0xA5)
        assert len(got) == len(want)
        for g, w in zip(got, want):
            assert g.size == w.size and np.array_equal(g, w), (tp, pp)
        back = O.reshard(m, O.Plan(tp, pp), O.Plan(1, 1), want, fill=0xA5)
        assert np.array_equal(back[0], full[0]), (tp, pp)


def test_any_plan_pair_against_np_split():
    sh, es = I.MICRO, 2
    m = model_of(sh)
    logical = npmodel.random_logical(sh, es, seed=5)
    images = {pl: npmodel.build_shards(sh, pl[0], pl[1], logical) for pl in plans_for(sh)}
    for a, b in itertools.product(images, images):
        got = O.reshard(m, O.Plan(*a), O.Plan(*b), images[a], fill=0xA5)
        for g, w in zip(got, images[b]):
            assert np.array_equal(g, w), (a, b)


def test_replicated_units_against_np_split():
    """k target units (a Split into k replica units, a weight sync to k units, Extend): unit r of the result is
    numpy's shard image of the target plan, for every r; with equal plans (Extend) every unit is the source image
    itself.  Target plans with pp > 1 and tp > 1 make a wrong unit stride land in the wrong buffer."""
    sh = I.MICRO
    m = model_of(sh)
    logical = npmodel.random_logical(sh, 2, seed=21)
    images = {pl: npmodel.build_shards(sh, pl[0], pl[1], logical) for pl in [(1, 1), (2, 2), (4, 2), (8, 1), (2, 4)]}
    for (a, b), k in itertools.product(itertools.product(images, images), (1, 2, 3)):
        got = O.reshard_replicated(m, O.Plan(*a), O.Plan(*b), k, images[a], fill=0xA5)
        n = b[0] * b[1]
        assert len(got) == k * n
        for r in range(k):
            for j in range(n):
                assert np.array_equal(got[r * n + j], images[b][j]), (a, b, k, r, j)
            if a == b:
                for j in range(n):
                    assert np.array_equal(got[r * n + j], images[a][j])


def test_state_with_optimizer_tensors_against_np_split():
    """(theta, omega): bf16 parameters and n_opt fp32 tensors of the parameters' layout, each with contents of
    its own, so that a slice of the buffer list taken at the wrong place, or a cast applied to omega, shows."""
    sh = I.MICRO
    m = model_of(sh)
    theta = npmodel.random_logical(sh, 2, seed=31)
    omega = [npmodel.random_logical(sh, 4, seed=32 + k) for k in range(3)]
    for a, b in [((2, 2), (4, 1)), ((4, 2), (1, 1)), ((1, 1), (2, 4)), ((8, 1), (8, 1))]:
        for n_opt in (0, 1, 3):
            src = npmodel.build_shards(sh, a[0], a[1], theta)
            want = npmodel.build_shards(sh, b[0], b[1], theta)
            for k in range(n_opt):
                src += npmodel.build_shards(sh, a[0], a[1], omega[k])
                want += npmodel.build_shards(sh, b[0], b[1], omega[k])
            got = O.reshard_state(m, O.Plan(*a), O.Plan(*b), n_opt, src, fill=0xA5)
            assert len(got) == len(want) == (1 + n_opt) * b[0] * b[1]
            for j, (g, w) in enumerate(zip(got, want)):
                assert g.size == w.size and np.array_equal(g, w), (a, b, n_opt, j)
    # omega stays fp32 when theta is cast: the parameters come out as torch's bf16 of the fp32 values
    m32 = model_of(sh, O.FP32)
    th32 = npmodel.random_logical(sh, 4, seed=41)
    src = npmodel.build_shards(sh, 2, 2, th32) + npmodel.build_shards(sh, 2, 2, omega[0])
    got = O.reshard_state(m32, O.Plan(2, 2), O.Plan(4, 1, O.BF16), 1, src, fill=0xA5)
    th16 = {n: O.rne_bf16_array(x).reshape(x.shape) for n, x in th32.items()}
    want = npmodel.build_shards(sh, 4, 1, th16) + npmodel.build_shards(sh, 4, 1, omega[0])
    for j, (g, w) in enumerate(zip(got, want)):
        assert np.array_equal(g, w), j


def test_more_distinct_parts_than_the_replica_record_holds_is_refused():
    sh = I.Shape(1, 1024, 128, 128, 256, 256)
    m = model_of(sh)
    src = [np.zeros(O.shard_bytes(m, O.Plan(128, 1), s), np.uint8) for s in range(128)]
    with pytest.raises(O.OracleError) as e:
        O.reshard(m, O.Plan(128, 1), O.Plan(1, 1), src)
    assert e.value.code == O.ERR_UNSUPPORTED


@pytest.mark.parametrize("sh", [I.TINY, I.MICRO])
def test_layout_variants_against_np(sh):
    """Grouped QKV and row-interleaved gate/up on either side: shards built by numpy (reshape to head groups,
    np.stack of the row sets) for every combination of source and target layout."""
    m = model_of(sh)
    logical = npmodel.random_logical(sh, 2, seed=31)
    pls = [p for p in plans_for(sh) if p in ((1, 1), (2, 1), (2, 2), (4, 2), (8, 1))]
    for la, lb in itertools.product(range(4), repeat=2):
        for a, b in itertools.product(pls, repeat=2):
            src = npmodel.build_shards(sh, a[0], a[1], logical, layout=la)
            want = npmodel.build_shards(sh, b[0], b[1], logical, layout=lb)
            got = O.reshard(m, O.Plan(a[0], a[1], 0, la), O.Plan(b[0], b[1], 0, lb), src, fill=0xA5)
            for g, w in zip(got, want):
                assert np.array_equal(g, w), (la, lb, a, b)


def test_layout_variant_sizes_and_cast():
    """The layout changes the order inside a rank's block, never what a rank holds: shard sizes are equal; the
    cast commutes with a layout conversion."""
    sh = I.SMALL
    m32 = model_of(sh, O.FP32)
    for pl in ((2, 2), (4, 1)):
        for lay in range(4):
            for s in range(pl[0] * pl[1]):
                assert O.shard_bytes(m32, O.Plan(pl[0], pl[1], 0, lay), s) == O.shard_bytes(m32, O.Plan(*pl), s)
    logical = npmodel.random_logical(sh, 4, seed=3)
    for n in logical:                                           # keep the fp32 payload finite and not NaN
        logical[n] = (logical[n] & np.uint32(0x3FFFFFFF)) | np.uint32(0x30000000)
    src = npmodel.build_shards(sh, 2, 2, logical, layout=3)     # Megatron-style training layout, fp32
    got = O.reshard(m32, O.Plan(2, 2, 0, 3), O.Plan(4, 1, O.BF16, 0), src, fill=0xA5)
    cast = {n: torch.from_numpy(x.view(np.float32)).to(torch.bfloat16).view(torch.int16).numpy().view(np.uint16)
            for n, x in logical.items()}
    for g, w in zip(got, npmodel.build_shards(sh, 4, 1, cast, layout=0)):
        assert np.array_equal(g, w)


def test_kv_head_replication_against_np():
    """tp > kv_heads: every kv head lives on tp/kv_heads ranks (np.split into heads, rank r takes head
    r // (tp/kv_heads)); q heads, FFN and vocabulary are cut as always.  Both directions and both QKV layouts."""
    sh = I.Shape(2, 128, 16, 2, 256, 256)                        # 16 q heads, 2 kv heads, head_dim 8
    m = model_of(sh)
    logical = npmodel.random_logical(sh, 2, seed=13)
    pls = [(1, 1), (2, 1), (4, 1), (8, 2), (16, 1)]
    for la, lb in [(0, 0), (1, 0), (0, 1), (3, 3)]:
        for a, b in itertools.product(pls, repeat=2):
            src = npmodel.build_shards(sh, a[0], a[1], logical, layout=la)
            want = npmodel.build_shards(sh, b[0], b[1], logical, layout=lb)
            got = O.reshard(m, O.Plan(a[0], a[1], 0, la), O.Plan(b[0], b[1], 0, lb), src, fill=0xA5)
            for g, w in zip(got, want):
                assert g.size == w.size and np.array_equal(g, w), (la, lb, a, b)
    assert O.check_plan(m, O.Plan(3, 1)) == O.ERR_INDIVISIBLE     # neither divides the other
    assert O.check_plan(m, O.Plan(32, 1)) == O.ERR_INDIVISIBLE    # more ranks than q heads
    src = npmodel.build_shards(sh, 8, 1, logical)
    p = O.locate(m, O.Plan(8, 1), 1, 3)                           # wk of layer 0 on rank 1: a copy of rank 0's head
    src[1][p.offset] ^= 1
    with pytest.raises(O.OracleError) as e:
        O.reshard(m, O.Plan(8, 1), O.Plan(1, 1), src)
    assert e.value.code == O.ERR_REPLICA_MISMATCH


def test_padded_vocabulary_against_np():
    """Vocabulary padded to a multiple of 128*tp before the cut (np.concatenate with filler rows, then np.split):
    the padding rows take room in the shards, are never read and never written, and V need not divide by tp."""
    sh = I.Shape(2, 64, 4, 4, 128, 1000)                         # V = 1000: divisible by neither 128 nor 3... by 1, 2, 4
    m = model_of(sh)
    logical = npmodel.random_logical(sh, 2, seed=17)
    assert O.check_plan(model_of(I.Shape(2, 64, 4, 4, 128, 1001)), O.Plan(2, 1)) == O.ERR_INDIVISIBLE
    assert O.check_plan(model_of(I.Shape(2, 64, 4, 4, 128, 1001)), O.Plan(2, 1, 0, 4)) == O.OK
    assert O.shard_bytes(m, O.Plan(4, 1, 0, 4), 0) > O.shard_bytes(m, O.Plan(4, 1), 0)      # 1024/4 vs 1000/4 rows
    cases = [((1, 1, 0), (4, 2, 4)), ((4, 2, 4), (1, 1, 0)), ((2, 1, 4), (4, 1, 4)), ((4, 1, 4), (2, 2, 0)),
             ((2, 2, 5), (4, 1, 6)), ((1, 2, 4), (1, 1, 4))]
    for (ta, pa, la), (tb, pb, lb) in cases:
        src = npmodel.build_shards(sh, ta, pa, logical, layout=la)
        want = npmodel.build_shards(sh, tb, pb, logical, layout=lb)
        got = O.reshard(m, O.Plan(ta, pa, 0, la), O.Plan(tb, pb, 0, lb), src, fill=0xA5)
        for g, w in zip(got, want):
            assert g.size == w.size and np.array_equal(g, w), ((ta, pa, la), (tb, pb, lb))
    odd = I.Shape(2, 64, 4, 4, 128, 1001)                        # only the padded cut can shard this vocabulary
    mo = model_of(odd)
    lo = npmodel.random_logical(odd, 2, seed=18)
    got = O.reshard(mo, O.Plan(1, 1), O.Plan(4, 1, 0, 4), npmodel.build_shards(odd, 1, 1, lo), fill=0xA5)
    for g, w in zip(got, npmodel.build_shards(odd, 4, 1, lo, layout=4)):
        assert np.array_equal(g, w)


def test_uneven_pipeline_cut_against_np():
    """pp that does not divide the layer count: the first L mod pp stages hold one layer more (np.array_split)."""
    sh = I.Shape(7, 64, 4, 4, 128, 256)
    m = model_of(sh)
    logical = npmodel.random_logical(sh, 2, seed=23)
    pls = [(1, 1), (2, 2), (1, 3), (4, 4), (2, 5), (1, 7)]
    assert O.check_plan(m, O.Plan(1, 8)) == O.ERR_INDIVISIBLE      # more stages than layers
    for a, b in itertools.product(pls, repeat=2):
        src = npmodel.build_shards(sh, a[0], a[1], logical)
        want = npmodel.build_shards(sh, b[0], b[1], logical)
        got = O.reshard(m, O.Plan(*a), O.Plan(*b), src, fill=0xA5)
        for g, w in zip(got, want):
            assert g.size == w.size and np.array_equal(g, w), (a, b)
    sizes = [O.shard_bytes(m, O.Plan(1, 3), s) for s in range(3)]   # 3 + 2 + 2 layers
    assert sizes[0] > sizes[1]


# ---------------------------------------------------------------- brute-force owner function

@pytest.mark.parametrize("es", [2, 4])
@pytest.mark.parametrize("vh", [False, True])
def test_owner_brute_force(es, vh):
    """Position-coded payload: every element of every logical tensor is looked up, one by one, through the
    per-element owner function in the shards the oracle produced."""
    sh = I.Shape(2, 32, 4, 2, 48, 64)
    m = model_of(sh, O.BF16 if es == 2 else O.FP32, vh)
    dt = npmodel.np_dtype(es)
    for salt in (1, 2, 3):
        logical = npmodel.position_coded(sh, es, salt, vh)
        src = npmodel.build_shards(sh, 1, 1, logical, vh)
        for tp, pp, lay in [(2, 1, 0), (1, 2, 0), (2, 2, 0), (2, 1, 3), (1, 1, 1), (2, 2, 2)]:
            dst = O.reshard(m, O.Plan(1, 1), O.Plan(tp, pp, 0, lay), src)
            seen = [np.zeros(d.size, np.uint8) for d in dst]
            for name, x in logical.items():
                for i in range(x.shape[0]):
                    for j in range(x.shape[1]):
                        for shard, off in npmodel.owner(sh, tp, pp, es, name, i, j, vh, lay):
                            assert dst[shard][off:off + es].view(dt)[0] == x[i, j], (name, i, j, tp, pp)
                            seen[shard][off:off + es] += 1
            for s, mask in enumerate(payload_mask(m, O.Plan(tp, pp))):
                assert np.array_equal(seen[s] == 1, mask)       # each payload byte owned exactly once


def test_owner_vectorised_tiny_merge():
    """The tiny Merge workload (TP2PP1 -> TP1PP1) checked through the owner function on sampled elements."""
    sh, es = I.TINY, 2
    m = model_of(sh)
    logical = npmodel.position_coded(sh, es, 7)
    src = npmodel.build_shards(sh, 2, 1, logical)
    dst = O.reshard(m, O.Plan(2, 1), O.Plan(1, 1), src)
    rng = np.random.default_rng(0)
    for name, x in logical.items():
        for _ in range(40):
            i, j = int(rng.integers(x.shape[0])), int(rng.integers(x.shape[1]))
            (shard, off), = npmodel.owner(sh, 1, 1, es, name, i, j)
            assert dst[shard][off:off + 2].view(np.uint16)[0] == x[i, j]
        for i, j in [(0, 0), (x.shape[0] - 1, x.shape[1] - 1)]:
            (shard, off), = npmodel.owner(sh, 1, 1, es, name, i, j)
            assert dst[shard][off:off + 2].view(np.uint16)[0] == x[i, j]


# ---------------------------------------------------------------- invariants

def _random_src(m, plan, seed, dtype):
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


def test_identity():
    for sh in (I.TINY, I.MICRO):
        m = model_of(sh)
        src = _random_src(m, O.Plan(1, 1), 0, "bf16")
        dst = O.reshard(m, O.Plan(1, 1), O.Plan(1, 1), src, fill=0xA5)
        mask = payload_mask(m, O.Plan(1, 1))[0]
        assert np.array_equal(dst[0][mask], src[0][mask])
        assert (dst[0][~mask] == 0xA5).all()


@pytest.mark.parametrize("sh", [I.TINY, I.SMALL])
def test_round_trip_all_plan_pairs(sh):
    m = model_of(sh)
    pls = plans_for(sh)
    for a in pls:
        src = _random_src(m, O.Plan(*a), 3, "bf16")
        masks = payload_mask(m, O.Plan(*a))
        for b in pls:
            mid = O.reshard(m, O.Plan(*a), O.Plan(*b), src)
            back = O.reshard(m, O.Plan(*b), O.Plan(*a), mid)
            for s, k, mk in zip(src, back, masks):
                assert np.array_equal(s[mk], k[mk]), (a, b)


def _checksums(m, plan, bufs):
    """Per logical tensor: (sum, xor) of element bit patterns over the shards' parts; replicated tensors
    divided by the replica count."""
    e = O.es(m, plan)
    dt = npmodel.np_dtype(e)
    out = []
    for t in range(O.num_logical(m)):
        rows, cols = O.logical_shape(m, t)
        tot, x, area = 0, 0, 0
        for s in range(len(bufs)):
            p = O.locate(m, plan, s, t)
            if p.held:
                v = bufs[s][p.offset:p.offset + p.nr * p.nc * e].view(dt).astype(np.uint64)
                tot += int(v.sum(dtype=np.uint64))
                x ^= int(np.bitwise_xor.reduce(v)) if (area // (rows * cols)) == 0 else 0
                area += p.nr * p.nc
        reps = area // (rows * cols)
        out.append(((tot // reps) % 2 ** 64, x))
    return out


def test_checksums_conserved():
    sh = I.TINY
    m = model_of(sh)
    src = _random_src(m, O.Plan(2, 1), 0, "bf16")       # the tiny Merge workload, seed 0
    ref = _checksums(m, O.Plan(2, 1), src)
    for b in plans_for(sh):
        dst = O.reshard(m, O.Plan(2, 1), O.Plan(*b), src)
        assert _checksums(m, O.Plan(*b), dst) == ref, b


def test_path_independence_paper_example():
    """(TP4, PP8) -> (TP8, PP2) directly equals the route through T_sub = (TP4, PP2), the paper's example of
    Section 6.1, and the route through the logical tensor (TP1, PP1)."""
    sh = I.MICRO
    m = model_of(sh)
    a, t_sub, c = O.Plan(4, 8), O.Plan(4, 2), O.Plan(8, 2)
    src = _random_src(m, a, 9, "bf16")
    direct = O.reshard(m, a, c, src)
    via_sub = O.reshard(m, t_sub, c, O.reshard(m, a, t_sub, src))
    via_one = O.reshard(m, O.Plan(1, 1), c, O.reshard(m, a, O.Plan(1, 1), src))
    for d, v, w in zip(direct, via_sub, via_one):
        assert np.array_equal(d, v) and np.array_equal(d, w)


def test_emu_example_tp1pp4_to_tp2pp4():
    """The EMU example of Section 5.1: an actor going from (TP1, PP4) to (TP2, PP4); checked against np.split."""
    sh = I.MICRO
    m = model_of(sh)
    logical = npmodel.random_logical(sh, 2, seed=21)
    got = O.reshard(m, O.Plan(1, 4), O.Plan(2, 4), npmodel.build_shards(sh, 1, 4, logical), fill=0xA5)
    for g, w in zip(got, npmodel.build_shards(sh, 2, 4, logical)):
        assert np.array_equal(g, w)


# ---------------------------------------------------------------- the cast

def _golden_cases():
    with open(os.path.join(GOLDEN, "rne_bf16_cases.txt")) as f:
        for line in f:
            line = line.strip()
            if line and not line.startswith("#"):
                a, b = line.split()[:2]
                yield int(a, 16), int(b, 16)


def test_cast_hand_cases():
    for u, want in _golden_cases():
        assert O.rne_bf16(u) == want, hex(u)


def test_cast_exact_nearest_on_samples():
    """Second formulation in exact integer arithmetic: the bf16 neighbours of a finite fp32 value are
    hi<<16 and (hi+1)<<16 read as sign-magnitude integers; choose the nearer, ties to the even hi."""
    rng = np.random.default_rng(1)
    us = np.concatenate([rng.integers(0, 2 ** 32, 20000, dtype=np.uint64),
                         np.arange(0x3F800000 - 70000, 0x3F800000 + 70000, 997, dtype=np.uint64)])
    for u in map(int, us):
        mag = u & 0x7FFFFFFF
        if mag > 0x7F800000:
            assert O.rne_bf16(u) == 0x7FC0
            continue
        lo = mag >> 16
        rem = mag - (lo << 16)
        if rem * 2 > 0x10000 or (rem * 2 == 0x10000 and lo & 1):
            lo += 1
        assert O.rne_bf16(u) == ((u >> 31) << 15 | lo), hex(u)


def test_cast_matches_torch_exhaustively():
    """Every one of the 2^32 fp32 bit patterns: equal to torch's fp32 -> bf16 conversion wherever the input is
    not NaN; every NaN gives 0x7FC0."""
    step = 1 << 24
    ramp = np.arange(step, dtype=np.uint32)
    for lo in range(0, 1 << 32, step):
        bits = ramp + np.uint32(lo)
        got = O.rne_bf16_array(bits)
        ref = torch.from_numpy(bits.view(np.float32)).to(torch.bfloat16).view(torch.int16).numpy().view(np.uint16)
        nan = (bits & 0x7FFFFFFF) > 0x7F800000
        assert np.array_equal(got[~nan], ref[~nan]), hex(lo)
        assert (got[nan] == 0x7FC0).all()


def test_cast_commutes_with_reshard():
    sh = I.TINY
    m32, m16 = model_of(sh, O.FP32), model_of(sh, O.BF16)
    a, b = O.Plan(2, 2), O.Plan(1, 1)
    src = _random_src(m32, a, 2, "fp32")
    fused = O.reshard(m32, a, O.Plan(b.tp, b.pp, O.BF16), src)
    # reshard in fp32, then cast the (TP1, PP1) image tensor by tensor with torch
    mid = O.reshard(m32, a, b, src)[0]
    want = np.zeros_like(fused[0])
    for t in range(O.num_logical(m32)):
        p32, p16 = O.locate(m32, b, 0, t), O.locate(m16, b, 0, t)
        n = p32.nr * p32.nc
        x = torch.from_numpy(mid[p32.offset:p32.offset + 4 * n].view(np.float32).copy())
        want[p16.offset:p16.offset + 2 * n] = x.to(torch.bfloat16).view(torch.int16).numpy().view(np.uint8)
    assert np.array_equal(fused[0], want)
    # cast first (shard by shard), then reshard in bf16
    a16 = []
    for s, buf in enumerate(src):
        out = np.zeros(O.shard_bytes(m16, a, s), np.uint8)
        for t in range(O.num_logical(m32)):
            p32, p16 = O.locate(m32, a, s, t), O.locate(m16, a, s, t)
            if p32.held:
                n = p32.nr * p32.nc
                out[p16.offset:p16.offset + 2 * n] = O.rne_bf16_array(
                    buf[p32.offset:p32.offset + 4 * n].view(np.uint32)).view(np.uint8)
        a16.append(out)
    assert np.array_equal(O.reshard(m16, a, b, a16)[0], fused[0])


# ---------------------------------------------------------------- refusals

def test_refusals():
    m = model_of(I.TINY)
    assert O.check_plan(m, O.Plan(4, 1)) == O.OK                    # tp > kv_heads: kv heads replicated
    assert O.check_plan(m, O.Plan(8, 1)) == O.ERR_INDIVISIBLE       # more ranks than q heads
    assert O.check_plan(m, O.Plan(1, 4)) == O.ERR_INDIVISIBLE       # 2 layers over 4 stages: a stage without a layer
    assert O.check_plan(model_of(I.Shape(2, 256, 4, 2, 689, 1024)), O.Plan(2, 1)) == O.ERR_INDIVISIBLE
    assert O.check_plan(m, O.Plan(0, 1)) == O.ERR_ARG
    src = _random_src(model_of(I.TINY, O.BF16), O.Plan(1, 1), 0, "bf16")
    with pytest.raises(O.OracleError) as e:                           # bf16 -> fp32 is not a transition
        O.reshard(m, O.Plan(1, 1), O.Plan(1, 1, O.FP32), src, O.new_shards(model_of(I.TINY, O.FP32), O.Plan(1, 1)))
    assert e.value.code == O.ERR_UNSUPPORTED


def test_replica_mismatch_is_detected():
    m = model_of(I.TINY)
    src = _random_src(m, O.Plan(2, 1), 0, "bf16")
    p = O.locate(m, O.Plan(2, 1), 1, 1)        # ln1 of layer 0 on TP rank 1
    src[1][p.offset] ^= 1
    with pytest.raises(O.OracleError) as e:
        O.reshard(m, O.Plan(2, 1), O.Plan(1, 1), src)
    assert e.value.code == O.ERR_REPLICA_MISMATCH
