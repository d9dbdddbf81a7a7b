"""Larger and odder shapes: Mixtral-shaped layers at full size (outputs sampled, the oracle
computes only the sampled down rows), a shape with more slices than warps, error codes."""
import ctypes

import numpy as np
import pytest
import torch

import oracle
from paper_2609_21137_b200 import synth

from helpers import (assert_output, assert_routing, bf16_tensor_to_f64, logit_gaps, MIN_LOGIT_GAP,
                     toolkit_for_specialisation)

pytestmark = pytest.mark.gpu


def _sampled_check(shp, rows, seed=0):
    from paper_2609_21137_b200 import binding
    for s in range(seed, seed + 10):
        layer = synth.make_layer(shp, seed=s)
        res = oracle.OracleLayer.from_synth(layer).decode_layer(layer.x, down_rows=rows)
        if logit_gaps(res, shp.k) > MIN_LOGIT_GAP or shp.k == shp.E:
            break
    mod = binding.MoeVqlrLayer.from_synth(layer, device="cuda")
    x = binding.bits_to_device(layer.x, "cuda")
    out, dbg = mod.decode(x, debug=True)
    torch.cuda.synchronize()
    assert_routing(dbg, res)
    got = bf16_tensor_to_f64(out)[:, rows]
    m = assert_output(got, res.out, what=shp.name)
    # the plain call is the one the benchmark times: at T = 1 it runs the expert kernel compiled for
    # this shape instead of the precompiled one that serves calls asking for the routing lists
    plain = mod.decode(x)
    torch.cuda.synchronize()
    assert torch.equal(plain.view(torch.int16), out.view(torch.int16))
    if toolkit_for_specialisation():
        assert mod.specialized() > 0, mod.specialization_note()
    mod.close()
    del layer
    return m


@pytest.mark.parametrize("mode", ["full", "paper"])
def test_mixtral_full_size_b1_sampled_rows(mode):
    shp = synth.shape("mixtral", mode=mode)
    rows = sorted(set(np.random.default_rng(1).integers(0, shp.H, 96).tolist()) | {0, shp.H - 1})
    _sampled_check(shp, rows)


@pytest.mark.parametrize("name,mode", [("mixtral_b4", "full"), ("mixtral_b4", "paper"),
                                       ("mixtral_b16", "full"), ("mixtral_b16", "paper")])
def test_mixtral_full_size_batches_sampled_rows(name, mode):
    # the named batch sizes at the named shape (I = 14336: 56 slices of the down contraction); the
    # oracle computes the sampled output rows of every (token, expert) pair
    shp = synth.shape(name, mode=mode)
    rows = sorted(set(np.random.default_rng(3).integers(0, shp.H, 48).tolist()) | {0, shp.H - 1})
    _sampled_check(shp, rows)


@pytest.mark.parametrize("name,mode", [("qwen3", "paper"), ("qwen3", "dense"), ("qwen3_b16", "paper"),
                                       ("dsv2lite", "paper"), ("dsv2lite_b8", "paper"),
                                       ("dsv2lite_deployed", "paper"), ("olmoe_deployed_b16", "paper")])
def test_named_configurations_at_their_own_expert_count(name, mode):
    # every output element against the oracle, with the models' E (128 / 64), bf16 down projection
    shp = synth.shape(name, mode=mode)
    rows = list(range(shp.H))
    _sampled_check(shp, rows)


@pytest.mark.parametrize("name", ["qwen3_b2", "qwen3_b4", "qwen3_b8"])
def test_batch_sizes_between_the_headline_points(name):
    # batch 2, 4 and 8 on the Qwen3 shape (all three projections compressed), sampled output rows
    shp = synth.shape(name)
    rows = sorted(set(np.random.default_rng(5).integers(0, shp.H, 96).tolist()) | {0, shp.H - 1})
    _sampled_check(shp, rows)


def test_more_slices_than_warps_b16():
    # I = 3584 -> 14 slices of the down contraction for 12 warps; every expert active at T = 16
    shp = synth.shape("mixtral_b16", I=3584)
    rows = sorted(set(np.random.default_rng(2).integers(0, shp.H, 64).tolist()) | {0, shp.H - 1})
    _sampled_check(shp, rows)


@pytest.mark.parametrize("name", ["qwen3_deployed", "qwen3_deployed_b16", "gemma4_deployed", "qwen3_3bit",
                                  "qwen3_5bit", "qwen3_d4_3bit", "qwen3_d4_4bit", "qwen3_d4_5bit"])
def test_papers_deployed_operating_points(name):
    # K = 256 / uint8, r = 384 (twelve low-rank parts), separate gate and up code books, bf16 down;
    # fewer experts than the real models to keep the oracle quick (routing width is unchanged)
    shp = synth.shape(name, E=24)
    layer, res = None, None
    for s in range(10):
        layer = synth.make_layer(shp, seed=s)
        res = oracle.OracleLayer.from_synth(layer).decode_layer(layer.x)
        if logit_gaps(res, shp.k) > MIN_LOGIT_GAP:
            break
    from paper_2609_21137_b200 import binding
    mod = binding.MoeVqlrLayer.from_synth(layer, device="cuda")
    out, dbg = mod.decode(binding.bits_to_device(layer.x, "cuda"), debug=True)
    torch.cuda.synchronize()
    assert_routing(dbg, res)
    assert_output(bf16_tensor_to_f64(out), res.out, what=name)
    plain = mod.decode(binding.bits_to_device(layer.x, "cuda"))
    torch.cuda.synchronize()
    assert torch.equal(plain.view(torch.int16), out.view(torch.int16))
    mod.close()


def test_host_buffer_entry_point_matches_device_path():
    from paper_2609_21137_b200 import binding
    shp = synth.shape("qwen3_b16", E=32)
    layer = synth.make_layer(shp, seed=0)
    mod = binding.MoeVqlrLayer.from_synth(layer, device="cuda")
    x = binding.bits_to_device(layer.x, "cuda")
    ref = mod.decode(x)
    torch.cuda.synchronize()
    xh = x.cpu().pin_memory()
    oh = torch.zeros((shp.T, shp.H), dtype=torch.int16).pin_memory()
    for _ in range(2):                     # the second call replays the captured graph
        oh.zero_()
        mod.decode_host(xh, oh)
        assert torch.equal(oh, ref.view(torch.int16).cpu())
    # fewer tokens than max_tokens through the same handle
    mod.decode_host(xh[:3].contiguous().pin_memory(), oh[:3])
    ref3 = mod.decode(x[:3].contiguous())
    torch.cuda.synchronize()
    assert torch.equal(oh[:3], ref3.view(torch.int16).cpu())
    mod.close()


def test_error_codes():
    from paper_2609_21137_b200 import binding
    layer = synth.make_layer(synth.shape("tiny", T=4), seed=0)
    mod = binding.MoeVqlrLayer.from_synth(layer, device="cuda", max_tokens=4)
    x = binding.bits_to_device(layer.x, "cuda")
    lib = binding.library()
    out = torch.empty((8, 256), dtype=torch.bfloat16, device="cuda")
    big = torch.zeros((8, 256), dtype=torch.bfloat16, device="cuda")
    st = ctypes.c_void_p(torch.cuda.current_stream().cuda_stream)
    assert lib.moe_vqlr_decode_layer(mod._h, big.data_ptr(), 5, out.data_ptr(), None, st) == binding.ERR_INVALID_ARG
    assert b"T=5" in lib.moe_vqlr_last_error(mod._h)
    assert lib.moe_vqlr_decode_layer(mod._h, big.data_ptr(), 0, out.data_ptr(), None, st) == binding.ERR_INVALID_ARG
    assert lib.moe_vqlr_decode_layer(mod._h, None, 1, out.data_ptr(), None, st) == binding.ERR_INVALID_ARG
    assert lib.moe_vqlr_decode_layer(mod._h, big.data_ptr() + 2, 1, out.data_ptr(), None, st) == binding.ERR_INVALID_ARG
    assert b"aligned" in lib.moe_vqlr_last_error(mod._h)
    mod.decode(x)                          # the handle still works after rejected calls
    torch.cuda.synchronize()
    mod.close()
    # unsupported shapes and options
    for kw, code in ((dict(d=2), binding.ERR_UNSUPPORTED), (dict(d=16), binding.ERR_UNSUPPORTED), (dict(max_tokens=17), binding.ERR_UNSUPPORTED),
                     (dict(k=9), binding.ERR_INVALID_ARG), (dict(H=260), binding.ERR_UNSUPPORTED)):
        with pytest.raises(binding.MoeVqlrError) as err:
            args = dict(H=256, I=128, E=8, k=2, S=0, d=8, K=256, r=16, max_tokens=4)
            args.update(kw)
            up = lambda a: binding.bits_to_device(a, "cuda")   # noqa: E731
            proj = lambda p: dict(codebook=up(p.codebook), idx=up(p.idx), basis=up(p.basis), factor=up(p.factor))  # noqa: E731
            binding.MoeVqlrLayer(router_w=up(layer.router_w), gate=proj(layer.gate), up=proj(layer.up),
                                 down=proj(layer.down), **args)
        assert err.value.status == code, kw


@pytest.mark.parametrize("d", [8, 4])
def test_index_validation_flag_finds_bad_index(d):
    from paper_2609_21137_b200 import binding
    layer = synth.make_layer(synth.shape("tiny", K=200, d=d), seed=0)
    binding.MoeVqlrLayer.from_synth(layer, device="cuda", flags=binding.FLAG_VALIDATE_INDICES).close()
    layer.up.idx[3, 7, layer.up.idx.shape[2] - 1] = 200      # the last index of a row: inside the scan for either d
    with pytest.raises(binding.MoeVqlrError) as err:
        binding.MoeVqlrLayer.from_synth(layer, device="cuda", flags=binding.FLAG_VALIDATE_INDICES)
    assert err.value.status == binding.ERR_BAD_INDEX
