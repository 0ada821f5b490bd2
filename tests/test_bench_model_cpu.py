"""The flop and byte models bench.py divides by: against the oracle's FLOP count (Appendix B) and against
hand-computed sizes, so that a roofline fraction cannot drift because a formula did."""
import os
import sys

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
sys.path.insert(0, ROOT)

import bench  # noqa: E402
from oracle import lory_oracle as O  # noqa: E402
from paper_2405_03133_b200.workloads import CONFIGS  # noqa: E402


@pytest.mark.parametrize("name", ["C2", "C3", "C4", "C5_T64", "C5_T1024"])
def test_layer_flops_match_the_oracle_count(name):
    wl = CONFIGS[name]
    assert bench.flops_per_step(wl) == O.layer_flops(wl.B, wl.L, wl.T, wl.d, wl.f, wl.E, backward=True)


def test_gemm_flops_add_up_to_the_ffn_part_of_the_layer():
    wl = CONFIGS["C3"]
    kf = bench.kernel_flops(wl)
    ffn = kf["gemm1_swiglu"] + kf["gemm2"] + kf["dh_dswiglu"] + 3 * kf["wgrad"] + kf["dx"]
    assert ffn == 3 * O.ffn_flops(wl.tokens, wl.d, wl.f)          # forward + backward = 3 x forward
    assert kf["merge"] == wl.S * O.merge_flops(wl.E, wl.d, wl.f)
    assert kf["stage2"] == 2 * kf["merge"]
    assert ffn + kf["merge"] + kf["stage2"] == bench.flops_per_step(wl)


def test_compulsory_bytes_at_c3():
    """What the method has to move: five activation tensors and three passes over the experts."""
    wl = CONFIGS["C3"]
    act = wl.tokens * wl.d * 2
    experts = wl.E * 3 * wl.d * wl.f * 2
    assert act == 67108864 and experts == 541065216
    assert bench.compulsory_bytes(wl) == 5 * act + 3 * experts
    assert 1.95e9 < bench.compulsory_bytes(wl) < 1.97e9
    # the parts of it each kernel touches add up to the whole: x twice more in the weight-gradient GEMMs and once
    # in the pooling on top of the five tensors, the experts three times
    mb = bench.method_bytes(wl)
    assert mb["merge"] == experts and mb["stage2"] == 2 * experts
    assert mb["gemm1_swiglu"] == mb["gemm2"] == mb["dh_dswiglu"] == mb["dx"] == mb["pool_router"] == act
    assert mb["wgrad"] == 2 * wl.tokens * (wl.d + wl.f)


def test_implementation_bytes_at_c3():
    """What this implementation moves on top: merged weights written once and read twice, their gradients written
    and read, the saved activations."""
    wl = CONFIGS["C3"]
    kb = bench.implementation_bytes(wl)
    P1 = wl.d * wl.f * 2                       # one bf16 matrix
    act_d, act_f = wl.tokens * wl.d * 2, wl.tokens * wl.f * 2
    assert kb["merge"] == 3 * (wl.E * P1 + wl.S * P1)
    assert kb["stage2"] == 3 * (wl.S * P1 + 2 * wl.E * P1)
    assert kb["gemm1_swiglu"] == act_d + 2 * wl.S * P1 + 3 * act_f
    assert kb["gemm2"] == act_f + wl.S * P1 + act_d
    assert kb["dh_dswiglu"] == act_d + wl.S * P1 + 4 * act_f
    assert kb["wgrad"] == act_d + act_f + wl.S * P1
    assert kb["dx"] == 2 * act_f + 2 * wl.S * P1 + act_d
    assert 15.0e9 < bench.implementation_bytes_per_step(wl) < 15.4e9
    assert 7.5 < bench.implementation_bytes_per_step(wl) / bench.compulsory_bytes(wl) < 7.9


def test_contractions_are_tensor_bound_and_streaming_kernels_hbm_bound():
    for k in ("gemm1_swiglu", "gemm2", "dh_dswiglu", "wgrad", "dx"):
        assert bench.KERNEL_BOUND[k] == "tensor"
    for k in ("merge", "stage2", "pool_router"):
        assert bench.KERNEL_BOUND[k] == "hbm"


def test_more_than_256_segments_cost_extra_expert_passes():
    wl = CONFIGS["C3"].with_(B=32)             # 512 segments: two launches of the merge and of its adjoint
    small = CONFIGS["C3"]
    P1 = wl.d * wl.f * 2
    assert bench.implementation_bytes(wl)["merge"] == 3 * (2 * wl.E * P1 + wl.S * P1)
    assert bench.implementation_bytes(wl)["stage2"] == 3 * (wl.S * P1 + 5 * wl.E * P1)
    assert bench.implementation_bytes(small)["merge"] == 3 * (small.E * P1 + small.S * P1)


def test_traffic_table_is_guarded_by_the_source_digest(monkeypatch):
    assert bench.measured_traffic("C2", "merge") is None        # only the captured workload has figures
    good = bench.NCU_TRAFFIC["C3"]["sources_sha1"]
    monkeypatch.setitem(bench.NCU_TRAFFIC["C3"], "sources_sha1", "0" * 40)
    assert bench.measured_traffic("C3", "merge") is None        # other sources: the figures no longer apply
    monkeypatch.setitem(bench.NCU_TRAFFIC["C3"], "sources_sha1", good)
