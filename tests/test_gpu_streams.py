"""The same layer through the other launch routes: a side stream (kernels chained by
programmatic dependent launch), a captured CUDA graph, and the generic kernels forced on a
shape the tensor-core kernels would normally take."""

import numpy as np
import pytest
import torch

from paper_2609_21137_b200 import synth

from helpers import assert_output, assert_routing, bf16_tensor_to_f64, make_checked_layer

pytestmark = pytest.mark.gpu

CASES = [synth.shape("tiny", T=3), synth.shape("qwen3", E=16), synth.shape("qwen3_b16", E=32),
         synth.shape("qwen3", E=16, mode="paper"), synth.shape("dsv2lite_b8", E=16),
         synth.shape("tiny", T=2, mode="dense")]


@pytest.mark.parametrize("shp", CASES, ids=lambda s: f"{s.name}-{s.mode}")
def test_side_stream_back_to_back(shp):
    from paper_2609_21137_b200 import binding
    layer, res, _ = make_checked_layer(shp, 0)
    mod = binding.MoeVqlrLayer.from_synth(layer, device="cuda")
    x = binding.bits_to_device(layer.x, "cuda")
    st = torch.cuda.Stream()
    torch.cuda.synchronize()
    with torch.cuda.stream(st):
        outs = [mod.decode(x, stream=st) for _ in range(3)]      # three chained calls
        out, dbg = mod.decode(x, debug=True, stream=st)
    st.synchronize()
    assert_routing(dbg, res)
    ref = bf16_tensor_to_f64(out)
    assert_output(ref, res.out)
    for o in outs:
        assert torch.equal(o.view(torch.int16), out.view(torch.int16))
    mod.close()


def test_graph_capture_replay():
    from paper_2609_21137_b200 import binding
    shapes = [synth.shape("qwen3", E=16), synth.shape("qwen3_b16", E=32, mode="paper")]
    mods, xs, outs, refs = [], [], [], []
    for shp in shapes:
        layer, res, _ = make_checked_layer(shp, 0)
        mods.append(binding.MoeVqlrLayer.from_synth(layer, device="cuda"))
        xs.append(binding.bits_to_device(layer.x, "cuda"))
        outs.append(torch.zeros((shp.T, shp.H), dtype=torch.bfloat16, device="cuda"))
        refs.append(res.out)
    graph = torch.cuda.CUDAGraph()
    torch.cuda.synchronize()
    with torch.cuda.graph(graph):
        for _ in range(2):
            for m, x, o in zip(mods, xs, outs):
                m.decode(x, out=o)
    for _ in range(2):
        for o in outs:
            o.zero_()
        graph.replay()
        torch.cuda.synchronize()
        for o, ref in zip(outs, refs):
            assert_output(bf16_tensor_to_f64(o), ref)
    for m in mods:
        m.close()


@pytest.mark.parametrize("shp", [synth.shape("tiny", T=5), synth.shape("qwen3", E=16, T=3, mode="paper")],
                         ids=lambda s: f"{s.name}-{s.mode}")
def test_generic_kernels_forced(shp):
    from paper_2609_21137_b200 import binding
    layer, res, _ = make_checked_layer(shp, 0)
    mod = binding.MoeVqlrLayer.from_synth(layer, device="cuda", flags=binding.FLAG_GENERIC_KERNELS)
    x = binding.bits_to_device(layer.x, "cuda")
    out, dbg = mod.decode(x, debug=True)
    torch.cuda.synchronize()
    assert_routing(dbg, res)
    assert_output(bf16_tensor_to_f64(out), res.out)
    mod.close()


@pytest.mark.parametrize("shp", [synth.shape("tiny", T=5), synth.shape("tiny", T=2, mode="paper"),
                                 synth.shape("qwen3", E=16, T=3), synth.shape("qwen3", E=16, T=9, mode="paper"),
                                 synth.shape("dsv2lite", E=16, T=1)],
                         ids=lambda s: f"{s.name}-{s.mode}-T{s.T}")
def test_persistent_kernel(shp):
    """MOE_VQLR_FLAG_PERSISTENT: the whole layer as one cooperative kernel gives the chain's results,
    in one launch per call, twice in a row (the grid barrier's state carries over between calls)."""
    from paper_2609_21137_b200 import binding
    layer, res, _ = make_checked_layer(shp, 0)
    mod = binding.MoeVqlrLayer.from_synth(layer, device="cuda", flags=binding.FLAG_PERSISTENT)
    x = binding.bits_to_device(layer.x, "cuda")
    for _ in range(2):
        before = mod.launch_count
        out, dbg = mod.decode(x, debug=True)
        torch.cuda.synchronize()
        assert mod.launch_count - before == 1
        assert_routing(dbg, res)
        assert_output(bf16_tensor_to_f64(out), res.out)
    mod.close()


@pytest.mark.parametrize("shp", [synth.shape("tiny", T=5), synth.shape("tiny", T=2, mode="paper"),
                                 synth.shape("qwen3", E=16, T=3), synth.shape("qwen3", E=16, T=9, mode="paper"),
                                 synth.shape("qwen3", E=16, T=16, I=832), synth.shape("dsv2lite", E=16, T=1),
                                 synth.shape("dsv2lite", E=16, T=2, mode="paper"),
                                 synth.shape("tiny", T=2, d=4), synth.shape("tiny", T=1, d=4, mode="paper"),
                                 synth.shape("olmoe_deployed", E=12, T=3), synth.shape("olmoe_deployed", E=12, T=1)],
                         ids=lambda s: f"{s.name}-{s.mode}-T{s.T}-I{s.I}-d{s.d}")
def test_fused_expert_kernel_forced(shp):
    """Router -> one kernel per (work group, slice of I) -> weighted sum, forced also where the
    items would not fill the GPU: three launches per call, the chain's results."""
    from paper_2609_21137_b200 import binding
    layer, res, _ = make_checked_layer(shp, 0)
    mod = binding.MoeVqlrLayer.from_synth(layer, device="cuda", flags=binding.FLAG_FORCE_FUSED)
    x = binding.bits_to_device(layer.x, "cuda")
    for _ in range(2):
        before = mod.launch_count
        out, dbg = mod.decode(x, debug=True)
        torch.cuda.synchronize()
        assert mod.launch_count - before == 3
        assert_routing(dbg, res)
        assert_output(bf16_tensor_to_f64(out), res.out)
    mod.close()


def test_fused_single_token_ties_and_no_renorm():
    """One token on the fused path: the blocks with an item find the selected experts by counting
    ranks, one other block by the k rounds of arg-max; both must follow the rule (logit descending,
    id ascending) when two router rows are identical, whichever side of the cut the pair falls on."""
    from paper_2609_21137_b200 import binding
    shp = synth.shape("tiny", T=1, E=8, k=3)
    for seed in range(8):
        for renorm in (True, False):
            layer, res, _ = make_checked_layer(shp, seed=seed, tie=(6, 2), renorm_topk=renorm)
            mod = binding.MoeVqlrLayer.from_synth(layer, device="cuda", renorm_topk=renorm,
                                                  flags=binding.FLAG_FORCE_FUSED)
            x = binding.bits_to_device(layer.x, "cuda")
            before = mod.launch_count
            out, dbg = mod.decode(x, debug=True)
            torch.cuda.synchronize()
            assert mod.launch_count - before == 3
            assert_routing(dbg, res)
            assert_output(bf16_tensor_to_f64(out), res.out)
            mod.close()


@pytest.mark.parametrize("shp", [
    synth.LayerShape("e70", H=512, I=256, E=70, k=5, d=8, K=700, r=16, T=1),            # E not a multiple of 4 or 32
    synth.LayerShape("e512", H=512, I=256, E=512, k=6, d=8, K=256, r=8, T=1, S=1),      # more experts than threads, replicated book
    synth.LayerShape("e70b", H=512, I=320, E=70, k=5, d=8, K=300, r=24, T=3, mode="paper", router_bias=True),
], ids=lambda s: s.name)
def test_fused_odd_expert_counts(shp):
    """The single-token routing of the fused path (rank by counting, ballots of 32 experts) on expert
    counts that do not fill its vector loads or its warps, and the forced multi-token path with a bias."""
    from paper_2609_21137_b200 import binding
    layer, res, _ = make_checked_layer(shp, 0)
    mod = binding.MoeVqlrLayer.from_synth(layer, device="cuda", flags=binding.FLAG_FORCE_FUSED)
    x = binding.bits_to_device(layer.x, "cuda")
    before = mod.launch_count
    out, dbg = mod.decode(x, debug=True)
    torch.cuda.synchronize()
    assert mod.launch_count - before == 3
    assert_routing(dbg, res)
    assert_output(bf16_tensor_to_f64(out), res.out)
    mod.close()


@pytest.mark.parametrize("mode", ["full", "paper"])
def test_fused_wide_slices(mode):
    """Slices of 15 row tiles (four k steps in the down product, the widest the fused kernel takes)."""
    from paper_2609_21137_b200 import binding
    shp = synth.LayerShape("wide_slices", H=512, I=2048, E=16, k=8, d=8, K=4096, r=64, T=1, mode=mode)
    layer, res, _ = make_checked_layer(shp, 0)
    mod = binding.MoeVqlrLayer.from_synth(layer, device="cuda")
    x = binding.bits_to_device(layer.x, "cuda")
    before = mod.launch_count
    out, dbg = mod.decode(x, debug=True)
    torch.cuda.synchronize()
    assert mod.launch_count - before == 3          # the fused path took it
    assert_routing(dbg, res)
    assert_output(bf16_tensor_to_f64(out), res.out)
    mod.close()


@pytest.mark.parametrize("mode", ["full", "paper"])
def test_one_handle_many_batch_sizes(mode):
    """One handle (max_tokens 16) serves calls of 1, 2, 5, 16 and again 1 tokens: the single-token
    calls take the fused path, the others the chain, on one workspace."""
    from paper_2609_21137_b200 import binding
    import oracle
    shp = synth.shape("qwen3", E=16, T=16, mode=mode)
    layer, _, _ = make_checked_layer(shp, 0)
    orc = oracle.OracleLayer.from_synth(layer)
    mod = binding.MoeVqlrLayer.from_synth(layer, device="cuda", max_tokens=16)
    for T in (1, 2, 5, 16, 1):
        res = orc.decode_layer(layer.x[:T])
        x = binding.bits_to_device(layer.x[:T], "cuda")
        before = mod.launch_count
        out, dbg = mod.decode(x, debug=True)
        torch.cuda.synchronize()
        assert mod.launch_count - before == (3 if T == 1 else 5)
        assert_routing(dbg, res)
        assert_output(bf16_tensor_to_f64(out), res.out)
    mod.close()


@pytest.mark.parametrize("shp", [synth.shape("tiny", T=1), synth.shape("tiny", T=5, mode="paper"),
                                 synth.shape("qwen3", E=16, T=1), synth.shape("dsv2lite", E=16, T=3),
                                 synth.shape("qwen3_deployed", E=24, T=2), synth.shape("qwen3", E=16, T=12)],
                         ids=lambda s: f"{s.name}-{s.mode}-T{s.T}")
def test_ablation_switches_keep_results(shp):
    """Section 5.4's mechanism switches: shared projections recomputed per expert, and one launch
    per work group for gate/up and down.  Both leave routing and outputs as they are; the launch
    count shows that the per-expert launches really happened."""
    from paper_2609_21137_b200 import binding
    layer, res, _ = make_checked_layer(shp, 0)
    x = binding.bits_to_device(layer.x, "cuda")
    n_pos = shp.T * (shp.k + shp.S)
    base = binding.MoeVqlrLayer.from_synth(layer, device="cuda")
    ref_out, _ = base.decode(x, debug=True)
    torch.cuda.synchronize()
    for flags in (binding.FLAG_ABLATE_Z_PER_EXPERT, binding.FLAG_ABLATE_PER_EXPERT_LAUNCH,
                  binding.FLAG_ABLATE_Z_PER_EXPERT | binding.FLAG_ABLATE_PER_EXPERT_LAUNCH):
        mod = binding.MoeVqlrLayer.from_synth(layer, device="cuda", flags=flags)
        for _ in range(2):
            before = mod.launch_count
            out, dbg = mod.decode(x, debug=True)
            torch.cuda.synchronize()
            launched = mod.launch_count - before
            assert_routing(dbg, res)
            assert_output(bf16_tensor_to_f64(out), res.out)
        if flags & binding.FLAG_ABLATE_PER_EXPERT_LAUNCH:
            assert launched >= 3 + 2 * n_pos, launched
        else:
            # same kernels, same summation order: bitwise the unswitched result
            assert torch.equal(out.view(torch.int16), ref_out.view(torch.int16))
        mod.close()
    base.close()


@pytest.mark.parametrize("shp", [synth.shape("tiny", T=5), synth.shape("tiny", T=2, mode="paper", K=100),
                                 synth.shape("dsv2lite", E=16, T=8), synth.shape("qwen3_deployed", E=24, T=16),
                                 synth.shape("dsv2lite", E=16, T=1), synth.shape("qwen3_deployed", E=24, T=1),
                                 synth.LayerShape("ragged_piece", H=8 * 48, I=128, E=6, k=2, S=1, d=8, K=256, r=40, T=3),
                                 synth.LayerShape("r0_books", H=1024, I=64, E=8, k=3, d=8, K=64, r=0, T=4,
                                                  per_projection_codebook=True)],
                         ids=lambda s: f"{s.name}-{s.mode}-T{s.T}")
def test_projection_code_book_path(shp):
    """MOE_VQLR_FLAG_PROJECTION_CODE_BOOK: gate/up through per-token tables T[b][k] = <x_b, codebook[k]> (Section 4.2)
    with the low-rank term in a kernel of its own: six launches per call, the oracle's results; one
    and several table pieces, a ragged piece, small code books, rank 0, separate books."""
    from paper_2609_21137_b200 import binding
    layer, res, _ = make_checked_layer(shp, 0)
    mod = binding.MoeVqlrLayer.from_synth(layer, device="cuda",
                                          flags=binding.FLAG_PROJECTION_CODE_BOOK | binding.FLAG_NO_FUSED)
    x = binding.bits_to_device(layer.x, "cuda")
    for _ in range(2):
        before = mod.launch_count
        out, dbg = mod.decode(x, debug=True)
        torch.cuda.synchronize()
        assert mod.launch_count - before == 6
        assert_routing(dbg, res)
        assert_output(bf16_tensor_to_f64(out), res.out)
    mod.close()


def test_two_live_handles_of_one_kernel_with_different_shared_memory_needs():
    """The shared-memory limit of a kernel belongs to the kernel, not to a handle: a second handle
    of the same shape with a smaller need (fewer tokens) must not lower it under the first one."""
    from paper_2609_21137_b200 import binding
    shp = synth.shape("qwen3_b16", E=32)
    layer, res, _ = make_checked_layer(shp, 0)
    big = binding.MoeVqlrLayer.from_synth(layer, device="cuda", max_tokens=16)
    small = binding.MoeVqlrLayer.from_synth(layer, device="cuda", max_tokens=1)     # same template instances
    x = binding.bits_to_device(layer.x, "cuda")
    out, dbg = big.decode(x, debug=True)            # would fail with ERR_CUDA if the limit had dropped
    torch.cuda.synchronize()
    assert_routing(dbg, res)
    assert_output(bf16_tensor_to_f64(out), res.out)
    out1 = small.decode(x[:1])
    torch.cuda.synchronize()
    assert torch.isfinite(out1.float()).all()
    small.close()
    big.close()


def test_bounded_wait_that_runs_out_is_reported_and_the_handle_recovers():
    """The persistent kernel's grid barrier is the library's only device-side spin.  With the test
    switch it waits for an arrival that never comes and gives up after 2000 polls: every block
    RETURNS (nothing traps, nothing hangs), the status word says MOE_VQLR_ERR_TIMEOUT, and the
    handle leaves the persistent kernel, so that the next call is correct."""
    from paper_2609_21137_b200 import binding
    shp = synth.shape("tiny", T=2)
    layer, res, _ = make_checked_layer(shp, 0)
    mod = binding.MoeVqlrLayer.from_synth(layer, device="cuda",
                                          flags=binding.FLAG_PERSISTENT | binding.FLAG_TEST_BARRIER_TIMEOUT)
    x = binding.bits_to_device(layer.x, "cuda")
    assert mod.last_status() == binding.OK
    before = mod.launch_count
    mod.decode(x)
    torch.cuda.synchronize()
    assert mod.launch_count - before == 1                  # it was the persistent kernel that ran
    assert mod.last_status() == binding.ERR_TIMEOUT
    assert mod.last_status() == binding.OK                 # reading clears it
    out, dbg = mod.decode(x, debug=True)                   # now the chain of kernels
    torch.cuda.synchronize()
    assert mod.last_status() == binding.OK
    assert_routing(dbg, res)
    assert_output(bf16_tensor_to_f64(out), res.out)
    # the host-buffer entry point reports the code by itself
    mod2 = binding.MoeVqlrLayer.from_synth(layer, device="cuda",
                                           flags=binding.FLAG_PERSISTENT | binding.FLAG_TEST_BARRIER_TIMEOUT)
    xh = x.cpu().pin_memory()
    oh = torch.empty((shp.T, shp.H), dtype=torch.bfloat16).pin_memory()
    with pytest.raises(binding.MoeVqlrError) as err:
        mod2.decode_host(xh, oh)
    assert err.value.status == binding.ERR_TIMEOUT
    mod2.decode_host(xh, oh)
    assert_output(bf16_tensor_to_f64(oh), res.out)
    # and a fresh handle is unaffected
    fresh = binding.MoeVqlrLayer.from_synth(layer, device="cuda", flags=binding.FLAG_PERSISTENT)
    out3 = fresh.decode(x)
    torch.cuda.synchronize()
    assert fresh.last_status() == binding.OK
    assert_output(bf16_tensor_to_f64(out3), res.out)
    for m in (mod, mod2, fresh):
        m.close()


@pytest.mark.parametrize("path", ["default", "generic"])
def test_non_finite_logits_are_reported(path):
    """A NaN in the tokens makes every router logit NaN: the ids stay in range and the status word
    reports MOE_VQLR_ERR_INVALID_ARG."""
    from paper_2609_21137_b200 import binding
    shp = synth.shape("tiny", T=2)
    layer, _, _ = make_checked_layer(shp, 0)
    mod = binding.MoeVqlrLayer.from_synth(layer, device="cuda",
                                          flags=binding.FLAG_GENERIC_KERNELS if path == "generic" else 0)
    xb = layer.x.copy()
    xb[1, 3] = 0x7FC0                                      # bf16 NaN in token 1
    x = binding.bits_to_device(xb, "cuda")
    _, dbg = mod.decode(x, debug=True)
    torch.cuda.synchronize()
    ids = dbg["topk_id"].cpu().numpy()
    assert ids.min() >= 0 and ids.max() < shp.E
    assert mod.last_status() == binding.ERR_INVALID_ARG
    mod.decode(binding.bits_to_device(layer.x, "cuda"))
    torch.cuda.synchronize()
    assert mod.last_status() == binding.OK
    mod.close()
