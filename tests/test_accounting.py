"""Byte accounting used by the benchmark: checked against the paper's own figures and against
the oracle's independent work counts."""
import oracle
from paper_2609_21137_b200 import accounting


def test_qwen3_dense_traffic_is_the_papers_75_mb():
    # Introduction: 8 of 128 experts, bf16 -> 75 MB of expert weights per layer per token
    assert abs(accounting.dense_equivalent_bytes(2048, 768, 8) / 1e6 - 75.5) < 0.1


def test_private_bytes_match_oracle_work_counts():
    for (H, I, d, K, r) in [(2048, 768, 8, 256, 384), (2048, 1408, 8, 256, 32), (4096, 14336, 8, 4096, 128)]:
        bJ = accounting.index_bits(K)
        wc = oracle.work_counts(H, I, d, K, r, b_J=bJ)
        per_proj = (wc["private_index_bits"] + wc["private_coeff_bits"]) / 8
        assert accounting.projection_private_bytes(True, I, H, d, K, r) == per_proj
        lb = accounting.layer_bytes(H=H, I=I, E=64, d=d, K=K, r=r, T=1, mode="paper", n_active=6)
        assert lb.per_expert_gateup == 2 * per_proj and lb.per_expert_down == 2 * H * I


def test_paper_operating_point_halves_the_expert_payload():
    # Section 5.2: with bf16 down, (8, 256, 384) on the Qwen3 shape reads exactly half the dense bytes
    lb = accounting.layer_bytes(H=2048, I=768, E=128, d=8, K=256, r=384, T=1, mode="paper", n_active=8)
    assert lb.per_expert * 2 == 3 * 2 * 2048 * 768


def test_layer_totals_for_the_benchmark_shapes():
    full = accounting.layer_bytes(H=2048, I=768, E=128, d=8, K=4096, r=64, T=1, mode="full", n_active=8)
    assert full.total == 524288 + 65536 + 2 * 262144 + 98304 + 8 * (983040 + 655360) + 8192
    paper = accounting.layer_bytes(H=2048, I=768, E=128, d=8, K=4096, r=64, T=1, mode="paper", n_active=8)
    assert paper.total == 524288 + 65536 + 2 * 262144 + 8 * (983040 + 2 * 2048 * 768) + 8192
    dense = accounting.layer_bytes(H=2048, I=768, E=128, d=8, K=4096, r=64, T=1, mode="dense", n_active=8)
    assert dense.total == 524288 + 8 * 3 * 2 * 2048 * 768 + 8192
    assert full.gateup_kernel == 8 * 983040 and full.down_kernel == 8 * 655360
