"""CUDA path against the fp64 oracle, element by element, through the C ABI."""
import numpy as np
import pytest
import torch

import oracle
from paper_2609_21137_b200 import synth

from helpers import (assert_output, assert_routing, bf16_tensor_to_f64, make_checked_layer,
                     run_gpu)

pytestmark = pytest.mark.gpu


def _full_check(shp, seed=0, **kw):
    layer, res, used = make_checked_layer(shp, seed)
    assert not res.bad_index
    mod, (out, dbg) = run_gpu(layer, **kw)
    assert_routing(dbg, res)
    m = assert_output(bf16_tensor_to_f64(out), res.out, what=f"{shp.name} seed {used}")
    mod.close()
    return m


@pytest.mark.parametrize("mode", ["full", "paper", "dense"])
def test_tiny(mode):
    _full_check(synth.shape("tiny", mode=mode))


@pytest.mark.parametrize("T", [1, 2, 3, 5, 8, 16])
def test_tiny_batches(T):
    _full_check(synth.shape("tiny", T=T, router_bias=True))


@pytest.mark.parametrize("mode", ["full", "paper"])
def test_ragged_shapes(mode):
    # H/8 and I/8 not multiples of eight blocks -> scalar index path; E not a multiple of 32;
    # r not a multiple of 32; several row tiles and a ragged tail of rows
    _full_check(synth.LayerShape("ragged", H=8 * 37, I=8 * 53, E=13, k=3, S=1, d=8, K=100, r=7,
                                 T=5, mode=mode))
    _full_check(synth.LayerShape("ragged16", H=8 * 40, I=8 * 72, E=70, k=5, d=8, K=700, r=33,
                                 T=7, mode=mode, router_bias=True))


def test_rank_zero_and_two_codebooks():
    _full_check(synth.LayerShape("r0", H=256, I=192, E=8, k=2, d=8, K=256, r=0, T=3))
    _full_check(synth.LayerShape("books", H=256, I=192, E=8, k=2, d=8, K=512, r=8, T=3,
                                 per_projection_codebook=True))


def test_more_rank_groups_than_slices():
    # the chain's gate/up kernel lets the slices carry the low-rank groups: two and three groups on
    # one slice (the third fetched late), uint16 and uint8 indices, four-value code words
    _full_check(synth.LayerShape("lr2_u16", H=256, I=192, E=8, k=2, d=8, K=512, r=64, T=3))
    _full_check(synth.LayerShape("lr3_u8", H=256, I=192, E=8, k=2, d=8, K=256, r=88, T=5, mode="paper"))
    _full_check(synth.LayerShape("lr2_d4", H=512, I=192, E=8, k=2, d=4, K=256, r=128, T=4))


def test_topk_equals_E_and_single_expert():
    _full_check(synth.LayerShape("kE", H=128, I=64, E=4, k=4, d=8, K=64, r=4, T=4))
    _full_check(synth.LayerShape("E1", H=128, I=64, E=1, k=1, d=8, K=64, r=4, T=2))


def test_exact_ties_go_to_lower_id():
    shp = synth.shape("tiny", T=16, E=8, k=3)
    layer, res, _ = make_checked_layer(shp, seed=0, tie=(6, 2))
    mod, (out, dbg) = run_gpu(layer)
    lg = dbg["logits"].cpu().numpy()
    assert np.array_equal(lg[:, 6], lg[:, 2])        # identical rows -> bitwise identical logits
    # the tie itself is exact on both sides; other gaps are far above fp32 error for this seed
    assert_routing(dbg, res)
    assert_output(bf16_tensor_to_f64(out), res.out)
    mod.close()


def test_no_renorm():
    shp = synth.shape("tiny", T=4)
    layer = synth.make_layer(shp, seed=0)
    res = oracle.OracleLayer.from_synth(layer, renorm_topk=False).decode_layer(layer.x)
    mod, (out, dbg) = run_gpu(layer, renorm_topk=False)
    assert_routing(dbg, res)
    assert_output(bf16_tensor_to_f64(out), res.out)
    mod.close()


def test_qwen3_b1():
    m = _full_check(synth.shape("qwen3"))
    assert m["norm_max"] < 1e-2


def test_qwen3_paper_and_dense_modes():
    _full_check(synth.shape("qwen3", mode="paper", E=16))
    _full_check(synth.shape("qwen3", mode="dense", E=16))


def test_qwen3_b16_grouping():
    _full_check(synth.shape("qwen3_b16"))


@pytest.mark.parametrize("name", ["dsv2lite", "dsv2lite_b8"])
def test_dsv2lite_shared_experts(name):
    _full_check(synth.shape(name))


def test_repeatable_bitwise():
    layer, res, _ = make_checked_layer(synth.shape("qwen3_b16", E=32), 0)
    mod, (out1, _) = run_gpu(layer)
    x = __import__("paper_2609_21137_b200.binding", fromlist=["x"]).bits_to_device(layer.x, "cuda")
    out2 = mod.decode(x)
    torch.cuda.synchronize()
    assert torch.equal(out1.view(torch.int16), out2.view(torch.int16))
    mod.close()


@pytest.mark.parametrize("path", ["default", "generic", "fused", "chain", "persistent"])
@pytest.mark.parametrize("shp", [synth.shape("tiny", T=1, act="gelu_tanh"),
                                 synth.shape("tiny", T=5, act="gelu_tanh", mode="paper"),
                                 synth.shape("qwen3", E=16, T=3, act="gelu_tanh")],
                         ids=lambda s: f"{s.name}-{s.mode}-T{s.T}")
def test_gelu_expert_activation(shp, path):
    """MOE_VQLR_FLAG_ACT_GELU_TANH on every kernel path (the generic kernels, the chain, the fused
    expert kernel, the persistent kernel): p = gelu_tanh(gate) * up as in the oracle; a path that
    ignored the flag would miss the tolerance (SiLU and GELU differ by 15 % at gate = 1)."""
    from paper_2609_21137_b200 import binding
    layer, res, _ = make_checked_layer(shp, 0)
    silu = oracle.OracleLayer.from_synth(layer, act="silu").decode_layer(layer.x)
    assert np.max(np.abs(silu.out - res.out)) > 0.05 * np.max(np.abs(res.out))
    flags = {"default": 0, "generic": binding.FLAG_GENERIC_KERNELS, "fused": binding.FLAG_FORCE_FUSED,
             "chain": binding.FLAG_NO_FUSED, "persistent": binding.FLAG_PERSISTENT}[path]
    mod, (out, dbg) = run_gpu(layer, flags=flags)
    assert_routing(dbg, res)
    assert_output(bf16_tensor_to_f64(out), res.out, what=f"{shp.name} gelu {path}")
    mod.close()


def test_gelu_long_intermediate():
    # I > 4096: the activation runs in the wide kernel of the chain
    shp = synth.LayerShape("longI", H=256, I=4608, E=4, k=2, d=8, K=256, r=16, T=2, act="gelu_tanh")
    _full_check(shp)


@pytest.mark.parametrize("shp", [synth.shape("tiny", d=4, T=1), synth.shape("tiny", d=4, T=5, mode="paper"),
                                 synth.LayerShape("ragged4", H=8 * 37, I=8 * 53, E=13, k=3, S=1, d=4, K=100, r=7, T=5),
                                 synth.LayerShape("books4", H=256, I=192, E=8, k=2, d=4, K=512, r=8, T=3,
                                                  per_projection_codebook=True),
                                 synth.LayerShape("olmoe_like", H=2048, I=1024, E=12, k=8, d=4, K=256, r=256,
                                                  T=4, mode="paper", per_projection_codebook=True),
                                 synth.LayerShape("olmoe_full", H=2048, I=1024, E=6, k=2, d=4, K=256, r=32, T=3)],
                         ids=lambda s: f"{s.name}-{s.mode}-T{s.T}")
def test_four_value_code_words(shp):
    """d = 4 (Section 5.5): code words of four values, two indices per eight weights; uint8 and
    uint16 indices, shared and separate code books, the shape of the paper's (4, 256, 256) point."""
    _full_check(shp)


def test_long_intermediate_many_pairs():
    # I > 4096 and many (token, expert) pairs: z_d comes from the kernel that takes four ranks per warp
    shp = synth.LayerShape("longI_b16", H=256, I=4608, E=6, k=3, d=8, K=256, r=128, T=16, router_bias=True)
    _full_check(shp)


@pytest.mark.parametrize("path", ["default", "generic", "fused", "chain", "persistent"])
@pytest.mark.parametrize("shp", [synth.shape("tiny", T=1, act="relu2"),
                                 synth.shape("tiny", T=5, act="relu2", mode="paper"),
                                 synth.shape("qwen3", E=16, T=3, act="relu2"),
                                 synth.shape("dsv2lite", E=16, T=1, act="relu2")],
                         ids=lambda s: f"{s.name}-{s.mode}-T{s.T}")
def test_up_only_relu2_experts(shp, path):
    """MOE_VQLR_FLAG_ACT_RELU2_UP_ONLY on every kernel path: experts without a gate projection,
    p = relu(W_up x)^2 (Section 5.7).  The tensor-core kernels skip the gate's bytes and products, the
    other paths repeat the up projection in its place; all must match the oracle, which never
    reads a gate."""
    from paper_2609_21137_b200 import binding
    layer, res, _ = make_checked_layer(shp, 0)
    assert layer.gate is None
    flags = {"default": 0, "generic": binding.FLAG_GENERIC_KERNELS, "fused": binding.FLAG_FORCE_FUSED,
             "chain": binding.FLAG_NO_FUSED, "persistent": binding.FLAG_PERSISTENT}[path]
    mod, (out, dbg) = run_gpu(layer, flags=flags)
    assert_routing(dbg, res)
    assert_output(bf16_tensor_to_f64(out), res.out, what=f"{shp.name} relu2 {path}")
    mod.close()


def test_nemotron_shaped_layer_and_a_padded_hidden_size():
    """The Nemotron-3-Nano-shaped layer at its deployed point (8, 256, 512): H = 2688, I = 1856,
    up-only ReLU^2 experts, bf16 down projection (fewer experts than the model to keep the oracle
    quick); and a hidden size that is not a multiple of the block length, padded by the caller with
    zero activations (the last four values of every token), as the paper's kernel does."""
    _full_check(synth.shape("nemotron_deployed", E=24))
    _full_check(synth.shape("nemotron_deployed", E=24, T=6))
    shp = synth.shape("nemotron_deployed", E=24, T=2, H=2688 + 64)       # "true" hidden size 2748, padded to 2752
    layer, _, _ = make_checked_layer(shp, 0)
    layer.x[:, 2748:] = 0
    res = oracle.OracleLayer.from_synth(layer).decode_layer(layer.x)
    mod, (out, dbg) = run_gpu(layer)
    assert_routing(dbg, res)
    assert_output(bf16_tensor_to_f64(out), res.out, what="padded hidden size")
    mod.close()


@pytest.mark.parametrize("path", ["default", "generic", "fused", "chain"])
@pytest.mark.parametrize("shp", [synth.shape("tiny", T=1, K=700, I=128, idx12=True),
                                 synth.shape("tiny", T=5, K=4096, mode="paper", idx12=True),
                                 synth.shape("qwen3", E=16, T=1, idx12=True),
                                 synth.shape("qwen3", E=16, T=9, idx12=True, act="relu2")],
                         ids=lambda s: f"{s.name}-{s.mode}-T{s.T}-K{s.K}")
def test_twelve_bit_packed_indices(shp, path):
    """MOE_VQLR_FLAG_IDX12: the index maps of all compressed projections packed to twelve bits.  The
    oracle reads the same packed bytes (and is pinned to give the uint16 layer's result bit for bit)."""
    from paper_2609_21137_b200 import binding
    layer, res, _ = make_checked_layer(shp, 0)
    assert layer.up.idx.dtype == np.uint8 and layer.up.idx.shape[-1] == (shp.H // 8) * 3 // 2
    flags = {"default": 0, "generic": binding.FLAG_GENERIC_KERNELS, "fused": binding.FLAG_FORCE_FUSED,
             "chain": binding.FLAG_NO_FUSED}[path]
    mod, (out, dbg) = run_gpu(layer, flags=flags)
    assert_routing(dbg, res)
    assert_output(bf16_tensor_to_f64(out), res.out, what=f"{shp.name} idx12 {path}")
    mod.close()


def test_twelve_bit_indices_limits_and_validation():
    from paper_2609_21137_b200 import binding
    # K = 256 has one-byte indices: the packed encoding is refused
    layer = synth.make_layer(synth.shape("tiny", K=700, I=128, idx12=True), 0)
    with pytest.raises(binding.MoeVqlrError) as err:
        binding.MoeVqlrLayer.from_synth(synth.Layer(shape=synth.shape("tiny", K=256, I=128, idx12=True), router_w=layer.router_w,
                                                    router_bias=None, x=layer.x, gate=layer.gate, up=layer.up, down=layer.down))
    assert err.value.status == binding.ERR_UNSUPPORTED
    # index validation unpacks the twelve-bit fields: 701 >= K = 700 is found
    packed = layer.up.idx
    bad = packed.copy()
    i0 = (700 + 1) & 0xFFF
    bad[1, 2, 0] = i0 & 0xFF
    bad[1, 2, 1] = (bad[1, 2, 1] & 0xF0) | (i0 >> 8)
    layer.up.idx = bad
    with pytest.raises(binding.MoeVqlrError) as err:
        binding.MoeVqlrLayer.from_synth(layer, flags=binding.FLAG_VALIDATE_INDICES)
    assert err.value.status == binding.ERR_BAD_INDEX
    layer.up.idx = packed
    binding.MoeVqlrLayer.from_synth(layer, flags=binding.FLAG_VALIDATE_INDICES).close()
