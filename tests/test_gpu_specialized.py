"""The single-token kernels compiled at create() for one layer shape (moe_vqlr_specialized):
they must exist on a box with the CUDA toolkit, run for plain single-token calls, and give
bitwise the results of the precompiled kernels (same source, same arithmetic order), which the
parity tests compare with the oracle."""
import pytest
import torch

from paper_2609_21137_b200 import synth
from tests.helpers import make_checked_layer, assert_output, bf16_tensor_to_f64, toolkit_for_specialisation

pytestmark = [pytest.mark.gpu,
              pytest.mark.skipif(not toolkit_for_specialisation(), reason="no NVRTC / CUDA headers: the precompiled kernels run")]

SHAPES = [
    synth.shape("qwen3", E=16),                                   # 16-bit indices, one 64 KB book, compressed down
    synth.shape("qwen3", E=16, mode="paper"),                     # dense bf16 down projection
    synth.shape("qwen3_deployed", E=16),                          # 8-bit indices, eight copies of the book
    synth.shape("dsv2lite", E=16),                                # shared experts
    synth.shape("qwen3_idx12", E=16),                             # 12-bit packed indices
    synth.shape("qwen3_d4_4bit", E=16),                           # four-value code words
    synth.shape("nemotron_deployed", E=16, H=1344, I=928),        # up-only experts (relu^2)
    synth.shape("qwen3", E=16, act="gelu_tanh"),
    synth.shape("tiny", T=1),
]


@pytest.mark.parametrize("T", [1, 6])
@pytest.mark.parametrize("shp", SHAPES, ids=lambda s: f"{s.name}-{s.mode}-{s.act}")
def test_specialised_equals_precompiled(shp, T):
    """T = 1: router -> fused expert kernel -> weighted sum, all three compiled per shape; T = 6: the
    chain, whose gate/up, down and weighted-sum kernels are."""
    from dataclasses import replace
    from paper_2609_21137_b200 import binding
    shp = replace(shp, T=T)
    layer, res, _ = make_checked_layer(shp, 0)
    x = binding.bits_to_device(layer.x, "cuda")
    spec = binding.MoeVqlrLayer.from_synth(layer, device="cuda")
    plain = binding.MoeVqlrLayer.from_synth(layer, device="cuda", flags=binding.FLAG_NO_SPECIALIZE)
    assert plain.specialized() == 0 and "NO_SPECIALIZE" in plain.specialization_note()
    assert spec.specialized() > 0, spec.specialization_note()      # every tensor-core configuration has at least the chain
    a = spec.decode(x)
    b = plain.decode(x)
    torch.cuda.synchronize()
    assert torch.equal(a.view(torch.int16), b.view(torch.int16))
    assert_output(bf16_tensor_to_f64(a), res.out, what=f"{shp.name} specialised T={T}")
    # repeated, and interleaved with a call that asks for the routing lists (at T = 1 that call runs
    # the precompiled expert kernel on the same handle)
    out_d, dbg = spec.decode(x, debug=True)
    c = spec.decode(x)
    torch.cuda.synchronize()
    assert torch.equal(out_d.view(torch.int16), a.view(torch.int16))
    assert torch.equal(c.view(torch.int16), a.view(torch.int16))
    assert spec.last_status() == 0
    spec.close()
    plain.close()


def test_headline_shape_is_specialised():
    """The benchmark's configuration must get its compiled copy on the GPU machine: a missing NVRTC or
    a compile error would otherwise only show as a slower layer."""
    from paper_2609_21137_b200 import binding, devsynth
    shp = synth.shape("qwen3")
    kw = devsynth.make_device_layer(shp, seed=0, device="cuda")
    kw.pop("x")
    mod = binding.MoeVqlrLayer(**kw)
    assert mod.specialized() == 3, mod.specialization_note()      # router, expert kernel, weighted sum (max_tokens = 1: no chain)
    mod.close()


def test_layers_of_one_shape_share_a_compilation():
    import time
    from paper_2609_21137_b200 import binding
    shp = synth.shape("qwen3", E=8, T=1)
    mods = []
    t = []
    for seed in range(3):
        layer, _, _ = make_checked_layer(shp, seed)
        t0 = time.perf_counter()
        mods.append(binding.MoeVqlrLayer.from_synth(layer, device="cuda"))
        t.append(time.perf_counter() - t0)
    assert all(m.specialized() == 3 for m in mods)
    assert t[2] < 0.5 * max(t[0], 0.5), t         # no second compilation (the first takes about a second)
    for m in mods:
        m.close()


ALLOWED_NOTES = ("do not run the fused kernel", "exceed one wave")


@pytest.mark.parametrize("mode", ["full", "paper", "dense"])
def test_every_named_workload_compiles_for_its_shape(mode):
    """Every workload of the tables, in every mode: the run-time compilation must succeed for its
    combination of index type, code-word length, code books, activation and work plan.  A compile
    error would otherwise only show as a slower layer (the precompiled kernels take over)."""
    from dataclasses import replace
    from paper_2609_21137_b200 import binding, devsynth
    seen = set()
    for name, shp in synth.SHAPES.items():
        key = (shp.H, shp.I, shp.k, shp.S, shp.d, shp.K, shp.r, shp.T, shp.act, shp.idx12, shp.per_projection_codebook, shp.router_bias)
        if key in seen or (shp.idx12 and mode == "dense"):
            continue
        seen.add(key)
        small = replace(shp, E=max(shp.k, min(shp.E, 8)), mode=mode)
        kw = devsynth.make_device_layer(small, seed=0, device="cuda")
        kw.pop("x")
        mod = binding.MoeVqlrLayer(**kw)
        note = mod.specialization_note()
        assert mod.specialized() > 0, f"{name} {mode}: {note}"
        assert note == "" or any(a in note for a in ALLOWED_NOTES), f"{name} {mode}: {note}"
        mod.close()
        del kw
        torch.cuda.empty_cache()


def _drawn_shapes(n, seed):
    """Shapes drawn from the ranges the tensor-core kernels cover (H a multiple of 64 so that rows
    split into whole groups of eight blocks), with the odd values that constant folding could get
    wrong: expert counts that are no multiple of 32, ranks that are no multiple of 32, a short
    last slice of I, shared experts, either index width, one or two code books, every activation."""
    import numpy as np
    rng = np.random.default_rng(seed)
    out = []
    for i in range(n):
        d = int(rng.choice([8, 8, 4]))
        K = int(rng.choice([64, 256] if d == 4 else [100, 256, 512, 1000, 4096]))
        if d == 4 and K % 2:
            K += 1
        mode = str(rng.choice(["full", "full", "paper"]))
        # a compressed down projection contracts over whole groups of eight blocks of I
        I = 64 * int(rng.integers(1, 13)) + (8 * int(rng.integers(0, 8)) if mode == "paper" else 0)
        out.append(synth.LayerShape(
            f"drawn{i}", H=64 * int(rng.integers(2, 20)), I=I,
            E=int(rng.integers(4, 41)), k=int(rng.integers(1, 5)), S=int(rng.choice([0, 0, 1, 2])), d=d, K=K,
            r=8 * int(rng.integers(0, 13)), T=int(rng.choice([1, 1, 2, 5, 9, 16])), router_bias=bool(rng.integers(0, 2)),
            mode=mode, per_projection_codebook=bool(rng.integers(0, 2)),
            act=str(rng.choice(["silu", "silu", "gelu_tanh", "relu2"]))))
    return out


@pytest.mark.parametrize("shp", _drawn_shapes(24, seed=20260921), ids=lambda s: f"{s.name}-H{s.H}-I{s.I}-E{s.E}-k{s.k}-S{s.S}-d{s.d}-K{s.K}-r{s.r}-T{s.T}-{s.mode}-{s.act}")
def test_drawn_shapes_specialised_equals_precompiled(shp):
    from paper_2609_21137_b200 import binding
    layer, res, _ = make_checked_layer(shp, 0)
    x = binding.bits_to_device(layer.x, "cuda")
    spec = binding.MoeVqlrLayer.from_synth(layer, device="cuda")
    plain = binding.MoeVqlrLayer.from_synth(layer, device="cuda", flags=binding.FLAG_NO_SPECIALIZE)
    note = spec.specialization_note()
    assert spec.specialized() > 0, note
    assert "nvrtc" not in note.lower(), note
    a = spec.decode(x)
    b = plain.decode(x)
    torch.cuda.synchronize()
    assert torch.equal(a.view(torch.int16), b.view(torch.int16))
    assert_output(bf16_tensor_to_f64(a), res.out, what=shp.name)
    assert spec.last_status() == 0
    spec.close()
    plain.close()


def test_toolkit_of_the_python_environment():
    """moe_vqlr_set_jit_toolkit: NVRTC and the CUDA headers from the nvidia-* packages of the Python
    environment instead of /usr/local/cuda give the same kernels (a new shape, so that it is compiled)."""
    from paper_2609_21137_b200 import binding
    nvrtc, inc = binding.pip_toolkit()
    if nvrtc is None:
        pytest.skip("no nvidia-cuda-nvrtc / nvidia-cuda-runtime packages in this environment")
    shp = synth.LayerShape("toolkit", H=512, I=320, E=12, k=3, d=8, K=256, r=24, T=1)
    layer, res, _ = make_checked_layer(shp, 0)
    x = binding.bits_to_device(layer.x, "cuda")
    binding.set_jit_toolkit(nvrtc, inc)
    try:
        mod = binding.MoeVqlrLayer.from_synth(layer, device="cuda")
        assert mod.specialized() > 0, mod.specialization_note()
        out = mod.decode(x)
        torch.cuda.synchronize()
        assert_output(bf16_tensor_to_f64(out), res.out, what="toolkit of the Python environment")
        mod.close()
    finally:
        binding.set_jit_toolkit(None, None)
