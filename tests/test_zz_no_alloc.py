"""The allocation-free routing entry point against the layer's own routing and the CPU oracle.

`moe_vqlr_route_noalloc` serves callers that are not allowed to allocate device memory (a
memory pool or the host application owns the device), so it keeps its logits in a fixed array
inside the library.  That array is shared by all calls and keeps old contents, which is why
the check is made on two calls in a row with different inputs: the second must not be affected
by what the first left behind.  Collected last on purpose (file name), so a failure here
cannot hide the results of the other GPU tests.
"""
import numpy as np
import pytest
import torch

from paper_2609_21137_b200 import synth

pytestmark = pytest.mark.gpu


def _layer_routing(layer):
    from paper_2609_21137_b200 import binding
    mod = binding.MoeVqlrLayer.from_synth(layer, device="cuda")
    x = binding.bits_to_device(layer.x, "cuda")
    _, dbg = mod.decode(x, debug=True)
    torch.cuda.synchronize()
    ids, w = dbg["topk_id"].cpu().numpy(), dbg["topk_w"].cpu().numpy()
    mod.close()
    return ids, w


def test_route_noalloc_matches_decode_layer_twice_in_a_row():
    from paper_2609_21137_b200 import binding
    # two different layers and batch sizes, the larger first so stale logits would be visible
    cases = [synth.make_layer(synth.shape("qwen3_b16", E=96), seed=1),
             synth.make_layer(synth.shape("tiny", T=3, router_bias=True), seed=2)]
    expected = [_layer_routing(layer) for layer in cases]
    # inputs and outputs are the caller's; allocate them all before the calls under test
    bufs = []
    for layer in cases:
        s = layer.shape
        bufs.append(dict(x=binding.bits_to_device(layer.x, "cuda"),
                         w=binding.bits_to_device(layer.router_w, "cuda"),
                         b=binding.bits_to_device(layer.router_bias, "cuda"),
                         ids=torch.full((s.T, s.k), -1, dtype=torch.int32, device="cuda"),
                         aff=torch.zeros((s.T, s.k), dtype=torch.float32, device="cuda")))
    torch.cuda.synchronize()
    for layer, buf in zip(cases, bufs):            # back to back on one stream
        rc = binding.route_noalloc(buf["x"], buf["w"], buf["b"], layer.shape.k, buf["ids"], buf["aff"])
        assert rc == binding.OK
    torch.cuda.synchronize()
    for buf, (ids, w) in zip(bufs, expected):
        np.testing.assert_array_equal(buf["ids"].cpu().numpy(), ids)
        np.testing.assert_allclose(buf["aff"].cpu().numpy(), w, rtol=0, atol=2e-6)


def _oracle_routing(layer, renorm=True):
    import oracle
    logits = oracle.OracleLayer.from_synth(layer, renorm_topk=renorm).router_logits(layer.x)
    return oracle.topk_affinity(logits, layer.shape.k, renorm)


@pytest.mark.parametrize("renorm", [True, False])
def test_route_noalloc_matches_the_oracle_and_allocates_nothing(renorm):
    """Against the CPU oracle's top-k and affinities (E = 72: not a multiple of 32 and more than
    32, so several words of the taken mask are in use), with the softmax over the selected k and
    over all E; and the free device memory is the same before and after the calls."""
    from paper_2609_21137_b200 import binding
    from helpers import make_checked_layer
    layer, _, _ = make_checked_layer(synth.shape("qwen3_b16", E=72, T=5), 3)
    ids_ref, w_ref = _oracle_routing(layer, renorm)
    s = layer.shape
    x = binding.bits_to_device(layer.x, "cuda")
    w = binding.bits_to_device(layer.router_w, "cuda")
    b = binding.bits_to_device(layer.router_bias, "cuda")
    ids = torch.full((s.T, s.k), -1, dtype=torch.int32, device="cuda")
    aff = torch.zeros((s.T, s.k), dtype=torch.float32, device="cuda")
    assert binding.route_noalloc(x, w, b, s.k, ids, aff, renorm_topk=renorm) == binding.OK      # resolves the array's address
    torch.cuda.synchronize()
    free0, _ = torch.cuda.mem_get_info()
    for _ in range(2):
        ids.fill_(-1)
        assert binding.route_noalloc(x, w, b, s.k, ids, aff, renorm_topk=renorm) == binding.OK
    torch.cuda.synchronize()
    free1, _ = torch.cuda.mem_get_info()
    assert free1 == free0, "the allocation-free entry point changed the free device memory"
    np.testing.assert_array_equal(ids.cpu().numpy(), ids_ref)
    np.testing.assert_allclose(aff.cpu().numpy(), w_ref, rtol=0, atol=2e-6)


def test_route_noalloc_rejects_sizes_beyond_its_fixed_scratch():
    from paper_2609_21137_b200 import binding
    x = torch.zeros((17, 64), dtype=torch.bfloat16, device="cuda")
    w = torch.zeros((8, 64), dtype=torch.bfloat16, device="cuda")
    ids = torch.zeros((17, 2), dtype=torch.int32, device="cuda")
    aff = torch.zeros((17, 2), dtype=torch.float32, device="cuda")
    assert binding.route_noalloc(x, w, None, 2, ids, aff) == binding.ERR_UNSUPPORTED      # T > 16
    w_big = torch.zeros((1025, 64), dtype=torch.bfloat16, device="cuda")
    assert binding.route_noalloc(x[:1], w_big, None, 2, ids, aff) == binding.ERR_UNSUPPORTED  # E > 1024
    assert binding.route_noalloc(x[:1], w, None, 9, ids, aff) == binding.ERR_INVALID_ARG   # k > E
    torch.cuda.synchronize()
