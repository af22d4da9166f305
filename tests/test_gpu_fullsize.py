"""Full-size parity of the benchmark workloads, in the launch configuration bench.py times.

Each workload is checked in two ways:
  * EVERY logical tensor (all 9L+3 of every model-stage) goes through the CPU oracle, from device slices of the
    sources, and is compared element by element with the device result (gpu_util.compare_every_tensor: the
    oracle call is the single-threaded routine as it stands; disjoint tensors run on a pool of host threads);
  * as a second line, a property that holds at any size: for every stored tensor the sum of its elements' bit
    patterns is the same on the source and the destination side (for the cast: the sum over torch's fp32 ->
    bf16 conversion of the source), and every replicated copy equals the first.
"""
import numpy as np
import pytest
import torch

import bench
import gpu_util as G
from oracle import oracle as O
from paper_2609_34645_b200 import binding as B
from paper_2609_34645_b200 import inputs as I

pytestmark = pytest.mark.gpu
ODT = {"bf16": O.BF16, "fp32": O.FP32}
TDT = {"bf16": torch.int16, "fp32": torch.int32}


def _need(bytes_needed):
    torch.cuda.empty_cache()                     # blocks cached from earlier tests count as used otherwise
    free, _ = torch.cuda.mem_get_info()
    if free < bytes_needed * 1.02 + (2 << 30):
        pytest.skip(f"needs {bytes_needed / 1e9:.1f} GB of device memory, {free / 1e9:.1f} GB free")


def _workload_bytes(name):
    tot = 0
    for st in I.WORKLOADS[name].stages:
        sh = st.shape
        d = B.ModelDesc(sh.layers, sh.hidden, sh.heads, sh.kv_heads, sh.ffn, sh.vocab, B.DTYPES[st.src[2]], st.value_head)
        tot += sum(d.shard_sizes(B.Plan(st.src[0], st.src[1], B.DTYPES[st.src[2]])))
        tot += sum(d.shard_sizes(B.Plan(st.dst[0], st.dst[1], B.DTYPES[st.dst[2]])))
    return tot


def _check_stage_sums(st, desc, src, dst, pa, pb, sdt, ddt):
    """Every stored tensor: element sums agree between the two sides; replicas agree with the first copy."""
    ses, des = I.element_size(sdt), I.element_size(ddt)
    for tid in range(desc.num_tensors()):
        want = None
        for s in range(desc.num_shards(pa)):
            off, rows, cols, rep = desc.tensor_slice(pa, s, tid)
            if not rows:
                continue
            x = src[s][off:off + rows * cols * ses]
            if sdt != ddt:
                v = x.view(torch.float32).to(torch.bfloat16).view(torch.int16).sum(dtype=torch.int64)
            else:
                v = x.view(TDT[sdt]).sum(dtype=torch.int64)
            if rep:
                want = v
                break
            want = v if want is None else want + v
        got, first = None, None
        for d in range(desc.num_shards(pb)):
            off, rows, cols, rep = desc.tensor_slice(pb, d, tid)
            if not rows:
                continue
            y = dst[d][off:off + rows * cols * des]
            v = y.view(TDT[ddt]).sum(dtype=torch.int64)
            if rep:
                if first is None:
                    first, got = y, v
                else:
                    assert torch.equal(first, y), f"replica of tensor {tid} differs on shard {d}"
            else:
                got = v if got is None else got + v
        assert int(want) == int(got), f"stage {st.name}: checksum of stored tensor {tid}"


def _run_workload(name):
    _need(_workload_bytes(name))
    wl, t, srcs, dsts, (parts, keep, descs) = bench.build_workload(name, torch.device("cuda"), dict(
        tile_bytes=0, ctas_per_sm=0, threads=0, variant=0))
    stream = torch.cuda.current_stream()
    t.run([b.data_ptr() for b in srcs], [b.data_ptr() for b in dsts], stream.cuda_stream)
    stream.synchronize()
    assert t.status() == B.DEV_OK
    return wl, t, srcs, dsts, descs


def oracle_job(st, src, dst_units, src_plan=None, dst_plan=None):
    """(model, source plan, target plan, sources, destination units) of one model-stage for
    gpu_util.compare_every_tensor, on the oracle's side of the fence."""
    sh = st.shape
    a, b = src_plan or st.src, dst_plan or st.dst
    m = O.Model(sh.layers, sh.hidden, sh.heads, sh.kv_heads, sh.ffn, sh.vocab, ODT[a[2]], st.value_head)
    return (m, O.Plan(a[0], a[1], 0, I.layout_of(a)), O.Plan(b[0], b[1], ODT[b[2]], I.layout_of(b)), src, dst_units)


def _check_plain_workload(name):
    wl, t, srcs, dsts, descs = _run_workload(name)
    si = di = 0
    jobs = []
    for st, (desc, pa, pb) in zip(wl.stages, descs):
        ns, nd = desc.num_shards(pa), desc.num_shards(pb)
        src, dst = srcs[si:si + ns], dsts[di:di + nd]
        si += ns
        di += nd
        _check_stage_sums(st, desc, src, dst, pa, pb, st.src[2], st.dst[2])
        jobs.append(oracle_job(st, src, [dst]))
    rd, wr = t.bytes()
    assert G.compare_every_tensor(jobs) == wr                 # every destination byte went through the oracle
    del srcs, dsts, src, dst, jobs
    torch.cuda.empty_cache()
    return rd, wr


def test_8b_identity_is_one_16gb_run():
    """Degenerate transition: equal plans collapse to a single contiguous run of 16 GB (the 8B shape has no
    padding), far beyond 32-bit byte offsets; the copy must be the identity."""
    sh = I.LLAMA_8B
    _need(2 * 16_060_522_496)
    d = B.ModelDesc(sh.layers, sh.hidden, sh.heads, sh.kv_heads, sh.ffn, sh.vocab, B.BF16)
    t = d.compile(B.Plan(1, 1), B.Plan(1, 1))
    assert len(t.rects()) == 1 and t.rects()[0].width_bytes_dst == 16_060_522_496
    src = I.make_shards(d.shard_sizes(B.Plan(1, 1)), "bf16", 99, "cuda")
    dst = I.sentinel_shards(d.shard_sizes(B.Plan(1, 1)), "cuda")
    stream = torch.cuda.current_stream()
    t.run([src[0].data_ptr()], [dst[0].data_ptr()], stream.cuda_stream)
    stream.synchronize()
    assert t.status() == B.DEV_OK
    assert torch.equal(src[0], dst[0])
    del src, dst
    torch.cuda.empty_cache()


def test_8b_split_tp1pp1_to_tp4pp2():
    rd, wr = _check_plain_workload("8b_tp1pp1_to_tp4pp2")
    assert rd == wr == 16_062_119_936


def test_8b_merge_tp4pp2_to_tp1pp1():
    rd, wr = _check_plain_workload("8b_tp4pp2_to_tp1pp1")
    assert rd == wr == 8_030_261_248 * 2


def test_8b_fp32_master_to_bf16_generation_layout():
    rd, wr = _check_plain_workload("8b_fp32_tp2pp2_to_bf16_tp4pp1")
    assert rd == 2 * wr


def test_ppo_five_stages_one_table():
    rd, wr = _check_plain_workload("ppo5_8b")
    assert rd == wr
    assert abs(rd + wr - 156.4e9) < 0.1e9


def test_32b_round_trip_into_the_sources():
    """TP2PP4 -> TP8PP1 -> TP2PP4 chained in one launch, the way back landing in the original source buffers
    (three 65.5 GB copies do not fit).  The chained run is checked on the middle layout (oracle samples, sums)
    and on the restored sources (recorded sums and slices).  Because a way back that wrote nothing would leave
    the sources looking right, the sources are then poisoned and the way back is run once more on its own."""
    name = "32b_tp2pp4_to_tp8pp1_and_back"
    _need(_workload_bytes(name))
    wl, t, srcs, dsts, (parts, keep, descs) = bench.build_workload(name, torch.device("cuda"), dict(
        tile_bytes=0, ctas_per_sm=0, threads=0, variant=0))
    st = wl.stages[0]
    desc, pa, pb = descs[0]
    ns, nd = desc.num_shards(pa), desc.num_shards(pb)
    mid = dsts[:nd]
    assert [b.data_ptr() for b in dsts[nd:]] == [b.data_ptr() for b in srcs]
    # keep sampled source slices (layer 0 and the last layer's wdown, final norm) to compare after the run
    sh = st.shape
    m = O.Model(sh.layers, sh.hidden, sh.heads, sh.kv_heads, sh.ffn, sh.vocab, O.BF16, False)
    opa = O.Plan(st.src[0], st.src[1])
    ids = list(range(1, 10)) + [9 * sh.layers, 9 * sh.layers + 1]
    kept = {}
    for tid in ids:
        for s in range(ns):
            p = O.locate(m, opa, s, tid)
            if p.held:
                kept[(tid, s)] = (p, srcs[s][p.offset:p.offset + p.nr * p.nc * 2].cpu().numpy().copy())
    sums = [b.view(torch.int16).sum(dtype=torch.int64).item() for b in srcs]
    stream = torch.cuda.current_stream()
    t.run([b.data_ptr() for b in srcs], [b.data_ptr() for b in dsts], stream.cuda_stream)
    stream.synchronize()
    assert t.status() == B.DEV_OK and t.num_tiles()[1] == 2
    # forward level against the oracle, every tensor (the sources hold the same bits again after the way back)
    _check_stage_sums(st, desc, srcs, mid, pa, pb, "bf16", "bf16")
    assert G.compare_every_tensor([oracle_job(st, srcs, [mid])]) == parts[0].bytes()[1]
    # the restored sources
    assert [b.view(torch.int16).sum(dtype=torch.int64).item() for b in srcs] == sums
    for (tid, s), (p, want) in kept.items():
        assert np.array_equal(srcs[s][p.offset:p.offset + want.size].cpu().numpy(), want), (tid, s)
    # poison the sources, then the way back alone must restore them from the middle layout
    for b in srcs:
        b.fill_(0x5A)
    back = parts[1]
    back.run([b.data_ptr() for b in mid], [b.data_ptr() for b in srcs], stream.cuda_stream)
    stream.synchronize()
    assert back.status() == B.DEV_OK
    assert [b.view(torch.int16).sum(dtype=torch.int64).item() for b in srcs] == sums
    for (tid, s), (p, want) in kept.items():
        assert np.array_equal(srcs[s][p.offset:p.offset + want.size].cpu().numpy(), want), (tid, s)
    # ... and the way back against the oracle, every tensor: middle layout -> original layout
    assert G.compare_every_tensor([oracle_job(st, mid, [srcs], st.dst, st.src)]) == parts[1].bytes()[1]
    rd, wr = t.bytes()
    assert abs(rd + wr - 2 * 131.05e9) < 0.3e9
    del srcs, dsts, mid
    torch.cuda.empty_cache()
