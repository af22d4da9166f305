"""Host-side pieces of bench.py that need no GPU: the memory a workload takes (the pre-flight of the workloads
measured after the headline) and the CPU-oracle legs (one core, and disjoint tensors on a pool of threads)."""
import bench
from oracle import oracle as O


def test_device_bytes_of_the_configurations():
    gb = {name: bench.workload_device_bytes(name) / 1e9 for name in bench.OTHER_CONFIGS + bench.OTHER_NEXT}
    assert abs(bench.workload_device_bytes(bench.DEFAULT_WORKLOAD) / 1e9 - 32.12) < 0.01
    assert abs(gb["tiny_tp2pp1_to_tp1pp1"] * 1e3 - 7.9) < 0.1
    assert abs(gb["8b_tp4pp2_to_tp1pp1"] - 32.12) < 0.01
    assert abs(gb["8b_fp32_tp2pp2_to_bf16_tp4pp1"] - 48.19) < 0.01
    assert abs(gb["ppo5_8b"] - 156.4) < 0.1                       # 78.2 GB of sources + 78.2 GB of destinations
    assert abs(gb["32b_tp2pp4_to_tp8pp1_and_back"] - 131.06) < 0.02     # the way back lands in the sources
    assert abs(gb["8b_extend_tp4pp2_x2"] - 3 * 16.06) < 0.05
    assert abs(gb["8b_state_adam_tp2pp2_to_tp4pp1"] - 5 * 32.12) < 0.1  # theta bf16 + two fp32 moments, both sides
    assert abs(gb["8b_dag_tp4pp8_to_tp8pp2"] - 6 * 16.06) < 0.1         # the source, four replicas, the target
    assert all(v < 170 for v in gb.values())                            # everything fits a 180 GB device


def test_oracle_legs_on_the_tiny_workload():
    O.build()
    one = bench.oracle_sample("tiny_tp2pp1_to_tp1pp1", 2, None, with_ends=True, workers=1)
    many = bench.oracle_sample("tiny_tp2pp1_to_tp1pp1", 2, None, with_ends=True, workers=4)
    for gbps, seconds, what in (one, many):
        assert gbps > 0 and seconds > 0
        assert "21 logical tensors" in what and "embedding" in what     # 9 x 2 layers + embed, final norm, head
    # the sample is the whole tiny workload: its bytes are the workload's
    assert "0.01 GB read+written of the workload's 0.01 GB" in one[2]
    assert bench.host_cores() >= 1
