"""GPU parity of the rows after the core path: k destination units (Extend; Split into replica units) and the
EMU's optimizer state, both through the C ABI against the oracle."""
import numpy as np
import pytest
import torch

import bench
import gpu_util as G
import test_gpu_fullsize as F
from oracle import oracle as O
from paper_2609_34645_b200 import binding as B
from paper_2609_34645_b200 import inputs as I

pytestmark = pytest.mark.gpu


@pytest.mark.parametrize("variant", [1, 2, 3])
@pytest.mark.parametrize("a,b,k,sdt,ddt", [((2, 2), (2, 2), 3, "bf16", "bf16"),      # Extend
                                           ((4, 1), (2, 2), 2, "bf16", "bf16"),      # Split into 2 replica units
                                           ((1, 1), (4, 2), 4, "bf16", "bf16"),
                                           ((2, 2), (4, 1), 2, "fp32", "bf16")])     # weight sync to 2 units
def test_replicated_destinations(a, b, k, sdt, ddt, variant):
    sh = I.SMALL
    desc = G.desc_of(sh, sdt)
    pa, pb = B.Plan(*a), B.Plan(b[0], b[1], B.DTYPES[ddt])
    for tile in (1024, 16384):
        t = desc.compile_replicated(pa, pb, k)
        t.tune(tile_bytes=tile, variant=variant)
        src = G.device_sources(desc, pa, sdt, 17)
        dst = G.Guarded([t.buffer_bytes(True, j) for j in range(t.num_buffers()[1])])
        G.run_transition(t, src, dst.bufs)
        want = O.reshard_replicated(G.omodel_of(sh, sdt), O.Plan(*a), O.Plan(b[0], b[1], G.ODT[ddt]), k,
                                    [s.cpu().numpy() for s in src], fill=G.SENTINEL)
        assert len(want) == len(dst.bufs) == k * b[0] * b[1]
        for g, w in zip(dst.bufs, want):
            assert np.array_equal(g.cpu().numpy(), w)
        assert dst.guards_intact()


@pytest.mark.parametrize("variant", [1, 2, 3])
def test_state_with_adam_moments(variant):
    sh = I.SMALL
    desc = G.desc_of(sh)
    a, b = (2, 2), (4, 1)
    pa, pb = B.Plan(*a), B.Plan(*b)
    t = desc.compile_state(pa, pb, 2)
    t.tune(variant=variant)
    p32 = B.Plan(a[0], a[1], B.FP32)
    src = G.device_sources(desc, pa, "bf16", 1) + G.device_sources(desc, p32, "fp32", 2) + \
        G.device_sources(desc, p32, "fp32", 3)
    dst = G.Guarded([t.buffer_bytes(True, j) for j in range(t.num_buffers()[1])])
    G.run_transition(t, src, dst.bufs)
    want = O.reshard_state(G.omodel_of(sh), O.Plan(*a), O.Plan(*b), 2, [s.cpu().numpy() for s in src],
                           fill=G.SENTINEL)
    for g, w in zip(dst.bufs, want):
        assert np.array_equal(g.cpu().numpy(), w)
    assert dst.guards_intact()


def _bytes_of(name):
    wl, t = I.WORKLOADS[name], None
    st = wl.stages[0]
    sh = st.shape
    d = B.ModelDesc(sh.layers, sh.hidden, sh.heads, sh.kv_heads, sh.ffn, sh.vocab, B.DTYPES[st.src[2]], st.value_head)
    pa = B.Plan(st.src[0], st.src[1], B.DTYPES[st.src[2]])
    pb = B.Plan(st.dst[0], st.dst[1], B.DTYPES[st.dst[2]])
    tot = sum(d.shard_sizes(pa)) + st.replicas * sum(d.shard_sizes(pb))
    tot += st.n_opt * (sum(d.shard_sizes(B.Plan(pa.tp, pa.pp, B.FP32))) + sum(d.shard_sizes(B.Plan(pb.tp, pb.pp, B.FP32))))
    return tot


def _run(name):
    F._need(_bytes_of(name))
    wl, t, srcs, dsts, (parts, keep, descs) = bench.build_workload(name, torch.device("cuda"), dict(
        tile_bytes=0, ctas_per_sm=0, threads=0, variant=0))
    stream = torch.cuda.current_stream()
    t.run([b.data_ptr() for b in srcs], [b.data_ptr() for b in dsts], stream.cuda_stream)
    stream.synchronize()
    assert t.status() == B.DEV_OK
    return wl, t, srcs, dsts, descs


def test_8b_extend_two_replicas_full_size():
    """Extend at full size: each new unit's shard equals the source shard, every byte (the 8B shape has no
    padding), which is the definition of a replica."""
    wl, t, srcs, dsts, descs = _run("8b_extend_tp4pp2_x2")
    n = len(srcs)
    assert len(dsts) == 2 * n
    for j, d in enumerate(dsts):
        assert torch.equal(d, srcs[j % n]), f"replica {j // n} shard {j % n}"
    rd, wr = t.bytes()
    assert wr == 2 * rd == 2 * sum(b.numel() for b in srcs)
    assert t.launch_info()["kernel"] == "nereus_walk_ring"
    del srcs, dsts
    torch.cuda.empty_cache()


def test_8b_weight_sync_to_two_generation_units_full_size():
    wl, t, srcs, dsts, descs = _run("8b_fp32_tp2pp2_to_bf16_tp4pp1_x2")
    st = wl.stages[0]
    desc, pa, pb = descs[0]
    n = desc.num_shards(pb)
    for j in range(n):
        assert torch.equal(dsts[j], dsts[n + j])                      # the two units are identical
    F._check_stage_sums(st, desc, srcs, dsts[:n], pa, pb, "fp32", "bf16")
    rd, wr = t.bytes()
    assert rd == wr                                                   # 4 B read, 2 x 2 B written per element
    assert G.compare_every_tensor([F.oracle_job(st, srcs, [dsts[:n], dsts[n:]])]) == wr   # every tensor, both units
    del srcs, dsts
    torch.cuda.empty_cache()


def test_8b_state_with_adam_full_size():
    wl, t, srcs, dsts, descs = _run("8b_state_adam_tp2pp2_to_tp4pp1")
    st = wl.stages[0]
    desc, pa, pb = descs[0]
    ns, nd = desc.num_shards(pa), desc.num_shards(pb)
    # parameters
    F._check_stage_sums(st, desc, srcs[:ns], dsts[:nd], pa, pb, "bf16", "bf16")
    jobs = [F.oracle_job(st, srcs[:ns], [dsts[:nd]])]
    # the two moments: fp32 on both sides, same (tp, pp)
    pa32, pb32 = B.Plan(pa.tp, pa.pp, B.FP32), B.Plan(pb.tp, pb.pp, B.FP32)
    st32 = I.Stage(st.name, st.shape, st.seed, (pa.tp, pa.pp, "fp32"), (pb.tp, pb.pp, "fp32"))
    d32 = B.ModelDesc(32, 4096, 32, 8, 14336, 128256, B.FP32)
    for k in range(2):
        s = srcs[ns * (1 + k):ns * (2 + k)]
        d = dsts[nd * (1 + k):nd * (2 + k)]
        F._check_stage_sums(st32, d32, s, d, pa32, pb32, "fp32", "fp32")
        jobs.append(F.oracle_job(st32, s, [d]))
    rd, wr = t.bytes()
    assert rd == wr == 5 * (8_030_261_248 * 2 + 65 * 8192 * 3)       # theta bf16 + two fp32 moments = 5x
    assert G.compare_every_tensor(jobs) == wr                         # every tensor of theta and of both moments
    del srcs, dsts, s, d
    torch.cuda.empty_cache()


def test_transition_estimate_predicts_the_measured_time():
    """L_tran from bytes and a bandwidth, held against CUDA-event time: with the bandwidth one workload
    measured (the 4-layer 8B Split), the estimate of another (its Merge back) is within 10% of its time."""
    def timed(name):
        wl, t, srcs, dsts, _ = bench.build_workload(name, torch.device("cuda"), dict(
            tile_bytes=0, ctas_per_sm=0, threads=0, variant=0))
        stream = torch.cuda.current_stream()
        sp, dp = [b.data_ptr() for b in srcs], [b.data_ptr() for b in dsts]
        for _ in range(3):
            t.run(sp, dp, stream.cuda_stream)
        a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        a.record(stream)
        for _ in range(5):
            t.run(sp, dp, stream.cuda_stream)
        b.record(stream)
        stream.synchronize()
        return t, a.elapsed_time(b) / 5 / 1e3
    t1, s1 = timed("8b4l_tp1pp1_to_tp4pp2")
    gbps = sum(t1.bytes()) / 1e9 / s1
    t2, s2 = timed("8b4l_tp4pp2_to_tp1pp1")
    assert t2.estimate(gbps, 0.0) == pytest.approx(s2, rel=0.10)
    torch.cuda.empty_cache()


@pytest.mark.parametrize("variant", [1, 2, 3])
@pytest.mark.parametrize("la,lb", [(3, 0), (0, 3), (1, 2), (3, 3)])
def test_layout_variants_on_the_gpu(la, lb, variant):
    """Grouped QKV / row-interleaved gate-up on either side, with and without the cast, both kernels."""
    sh = I.SMALL
    for sdt, ddt, a, b in [("bf16", "bf16", (2, 2), (4, 1)), ("fp32", "bf16", (4, 1), (2, 2))]:
        desc = G.desc_of(sh, sdt)
        pa, pb = B.Plan(a[0], a[1], 0, la), B.Plan(b[0], b[1], B.DTYPES[ddt], lb)
        t = desc.compile(pa, pb)
        t.tune(variant=variant, tile_bytes=4096)
        src = G.device_sources(desc, pa, sdt, 23)
        dst = G.Guarded([t.buffer_bytes(True, j) for j in range(t.num_buffers()[1])])
        G.run_transition(t, src, dst.bufs)
        want = O.reshard(G.omodel_of(sh, sdt), O.Plan(a[0], a[1], 0, la), O.Plan(b[0], b[1], G.ODT[ddt], lb),
                         [s.cpu().numpy() for s in src], fill=G.SENTINEL)
        for g, w in zip(dst.bufs, want):
            assert np.array_equal(g.cpu().numpy(), w)
        assert dst.guards_intact()


def test_8b_trainer_layout_to_generation_layout_full_size():
    """fp32 weights in a trainer's layout (grouped QKV, interleaved gate/up, TP2PP2) to blocked bf16 TP4PP1:
    every tensor against the oracle, and the sums of all stored tensors."""
    name = "8b_grouped_fp32_tp2pp2_to_blocked_bf16_tp4pp1"
    wl, t, srcs, dsts, descs = _run(name)
    st = wl.stages[0]
    desc, pa, pb = descs[0]
    F._check_stage_sums(st, desc, srcs, dsts, pa, pb, "fp32", "bf16")
    # every tensor through the oracle; under the grouped and interleaved layouts a part's rows are interleaved
    # with other tensors' rows, which the comparison handles by the span of each part
    G.compare_every_tensor([F.oracle_job(st, srcs, [dsts])])
    del srcs, dsts
    torch.cuda.empty_cache()


@pytest.mark.parametrize("variant", [1, 2])
def test_lowered_dag_runs_in_one_launch(variant):
    """The paper's (TP4, PP8) -> (TP8, PP2) example planned as Split / Destroy / Merge, lowered to one table with
    two dependency levels and run in one launch: replicas and target against the oracle."""
    from oracle import dag_rules as D
    from test_dag_cpu import U, lowered
    sh = I.MICRO
    dag, t, descs = lowered([D.StageChange(D.INFERENCE, [U(4, 8, 0)], [U(8, 2, 0)])], [sh])
    t.tune(variant=variant, tile_bytes=2048)
    src = G.device_sources(descs[0], B.Plan(4, 8), "bf16", 3)
    n_src, n_dst = t.num_buffers()
    dst = G.Guarded([t.buffer_bytes(True, j) for j in range(n_dst)])
    G.run_transition(t, src, dst.bufs)
    assert t.launches() == 1 and t.num_tiles()[1] == 2
    host = [s.cpu().numpy() for s in src]
    m = G.omodel_of(sh)
    sub = O.reshard(m, O.Plan(4, 8), O.Plan(4, 2), host, fill=G.SENTINEL)
    for k in range(4):
        for g, w in zip(dst.bufs[8 * k:8 * k + 8], sub):
            assert np.array_equal(g.cpu().numpy(), w)
    for g, w in zip(dst.bufs[32:], O.reshard(m, O.Plan(4, 8), O.Plan(8, 2), host, fill=G.SENTINEL)):
        assert np.array_equal(g.cpu().numpy(), w)
    assert dst.guards_intact()


def test_8b_dag_full_size():
    name = "8b_dag_tp4pp8_to_tp8pp2"
    F._need(96 * (1 << 30))
    wl, t, srcs, dsts, extra = bench.build_workload(name, torch.device("cuda"), dict(
        tile_bytes=0, ctas_per_sm=0, threads=0, variant=0))
    stream = torch.cuda.current_stream()
    t.run([b.data_ptr() for b in srcs], [b.data_ptr() for b in dsts], stream.cuda_stream)
    stream.synchronize()
    assert t.status() == B.DEV_OK and t.num_tiles()[1] == 2
    assert len(srcs) == 32 and len(dsts) == 4 * 8 + 16
    for k in range(1, 4):                                     # the four replicas are identical
        for a, b in zip(dsts[0:8], dsts[8 * k:8 * k + 8]):
            assert torch.equal(a, b)
    st = wl.stages[0]
    desc = extra[1][0]
    F._check_stage_sums(st, desc, srcs, dsts[32:], B.Plan(4, 8), B.Plan(8, 2), "bf16", "bf16")
    F._check_stage_sums(st, desc, srcs, dsts[:8], B.Plan(4, 8), B.Plan(4, 2), "bf16", "bf16")
    # every tensor through the oracle: the first replica against (TP4,PP8)->(TP4,PP2) (the other three equal it,
    # checked above), the target against the direct (TP4,PP8)->(TP8,PP2)
    G.compare_every_tensor([F.oracle_job(st, srcs, [dsts[:8]], (4, 8, "bf16"), (4, 2, "bf16")),
                            F.oracle_job(st, srcs, [dsts[32:]], (4, 8, "bf16"), (8, 2, "bf16"))])
    del srcs, dsts
    torch.cuda.empty_cache()


GQA16 = I.Shape(2, 128, 16, 2, 256, 256)          # 16 q heads, 2 kv heads, head_dim 8


@pytest.mark.parametrize("variant", [1, 2, 3])
@pytest.mark.parametrize("a,b", [((1, 1), (8, 1)), ((8, 2), (2, 1)), ((16, 1), (4, 2)), ((4, 1), (16, 1))])
def test_kv_head_replication_on_the_gpu(a, b, variant):
    """tp > kv_heads on either side, bit copy and cast, both kernels."""
    for sdt, ddt, la, lb in [("bf16", "bf16", 0, 0), ("fp32", "bf16", 1, 0)]:
        desc = G.desc_of(GQA16, sdt)
        pa, pb = B.Plan(a[0], a[1], 0, la), B.Plan(b[0], b[1], B.DTYPES[ddt], lb)
        t = desc.compile(pa, pb)
        t.tune(variant=variant, tile_bytes=1024)
        src = G.device_sources_by_oracle(GQA16, O.Plan(a[0], a[1], 0, la), sdt, 29)
        dst = G.Guarded([t.buffer_bytes(True, j) for j in range(t.num_buffers()[1])])
        G.run_transition(t, src, dst.bufs)
        want = O.reshard(G.omodel_of(GQA16, sdt), O.Plan(a[0], a[1], 0, la), O.Plan(b[0], b[1], G.ODT[ddt], lb),
                         [s.cpu().numpy() for s in src], fill=G.SENTINEL)
        for g, w in zip(dst.bufs, want):
            assert np.array_equal(g.cpu().numpy(), w)
        assert dst.guards_intact()


def test_8b_tp16_beyond_the_kv_heads_full_size():
    wl, t, srcs, dsts, descs = _run("8b_tp4pp1_to_tp16pp1")
    st = wl.stages[0]
    desc, pa, pb = descs[0]
    G.compare_every_tensor([F.oracle_job(st, srcs, [dsts])])          # every tensor through the oracle
    # kv heads: ranks 2g and 2g+1 hold the same K and V rows of every layer
    for tid in (1 + 6 * 0 + 1, 1 + 6 * 31 + 1):
        off, rows, cols, _ = desc.tensor_slice(pb, 0, tid)
        q_rows = 32 * 128 // 16
        for r in range(0, 16, 2):
            a = dsts[r][off + q_rows * cols * 2: off + rows * cols * 2]
            b = dsts[r + 1][off + q_rows * cols * 2: off + rows * cols * 2]
            assert torch.equal(a, b)
    rd, wr = t.bytes()
    assert rd == wr > 8_030_261_248 * 2 + 16 * 65 * 8192         # replicated kv heads move once per holder
    del srcs, dsts
    torch.cuda.empty_cache()


@pytest.mark.parametrize("variant", [1, 2, 3])
def test_mixed_cast_and_copy_table(variant):
    """One table with cast tiles (fp32 parameters -> bf16) and bit-copy tiles (fp32 optimizer moments): the
    converting ring serves both kinds."""
    sh = I.SMALL
    desc = G.desc_of(sh, "fp32")
    a, b = (2, 2), (4, 1)
    pa, pb = B.Plan(a[0], a[1], B.FP32), B.Plan(b[0], b[1], B.BF16)
    t = desc.compile_state(pa, pb, 2)
    assert {r.cast for r in t.rects()} == {0, 1}
    t.tune(variant=variant, tile_bytes=4096)
    assert t.launch_info()["kernel"] == {1: "nereus_walk_vec", 2: "nereus_walk_ring", 3: "nereus_walk_once"}[variant]
    src = G.device_sources(desc, pa, "fp32", 1) + G.device_sources(desc, pa, "fp32", 2) + \
        G.device_sources(desc, pa, "fp32", 3)
    dst = G.Guarded([t.buffer_bytes(True, j) for j in range(t.num_buffers()[1])])
    G.run_transition(t, src, dst.bufs)
    want = O.reshard_state(G.omodel_of(sh, "fp32"), O.Plan(*a), O.Plan(b[0], b[1], O.BF16), 2,
                           [s.cpu().numpy() for s in src], fill=G.SENTINEL)
    for g, w in zip(dst.bufs, want):
        assert np.array_equal(g.cpu().numpy(), w)
    assert dst.guards_intact()


@pytest.mark.parametrize("variant", [1, 2, 3])
def test_padded_vocabulary_on_the_gpu(variant):
    """Vocabulary padded to a multiple of 128*tp on either side: padding rows stay as they were (sentinel)."""
    sh = I.Shape(2, 64, 4, 4, 128, 1000)
    for (a, la), (b, lb), sdt, ddt in [(((1, 1), 0), ((4, 2), 4), "bf16", "bf16"),
                                       (((4, 2), 4), ((2, 1), 0), "bf16", "bf16"),
                                       (((2, 1), 4), ((4, 1), 4), "fp32", "bf16"),
                                       (((4, 1), 5), ((2, 2), 6), "fp32", "fp32")]:
        desc = G.desc_of(sh, sdt)
        pa, pb = B.Plan(a[0], a[1], 0, la), B.Plan(b[0], b[1], B.DTYPES[ddt], lb)
        t = desc.compile(pa, pb)
        t.tune(variant=variant, tile_bytes=1024)
        src = G.device_sources_by_oracle(sh, O.Plan(a[0], a[1], 0, la), sdt, 41)
        dst = G.Guarded([t.buffer_bytes(True, j) for j in range(t.num_buffers()[1])])
        G.run_transition(t, src, dst.bufs)
        want = O.reshard(G.omodel_of(sh, sdt), O.Plan(a[0], a[1], 0, la), O.Plan(b[0], b[1], G.ODT[ddt], lb),
                         [s.cpu().numpy() for s in src], fill=G.SENTINEL)
        for g, w in zip(dst.bufs, want):
            assert np.array_equal(g.cpu().numpy(), w)
        assert dst.guards_intact()
