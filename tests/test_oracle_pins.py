"""Pins for the CPU oracle: each test ties one part of it to something outside itself — a
value the paper prints, a brute-force evaluation in the paper's own index order, a closed
form, an invariant, or a library routine (numpy / torch fp64)."""
import itertools
import os

import numpy as np
import pytest
import torch

import oracle
from paper_2609_21137_b200 import synth

GOLDEN = os.path.join(os.path.dirname(__file__), "golden", "paper_printed_values.txt")


def f64(bits):
    return synth.bf16_bits_to_f64(bits)


def small_shape(**kw):
    base = dict(name="t", H=48, I=24, E=6, k=2, S=0, d=8, K=32, r=4, T=3, mode="full")
    base.update(kw)
    return synth.LayerShape(**base)


# ------------------------------------------------------------------------------------------
# accounting against values printed in the paper
# ------------------------------------------------------------------------------------------
def _golden_rows():
    rows = []
    for line in open(GOLDEN):
        line = line.strip()
        if not line or line.startswith("#"):
            continue
        f = [c.strip() for c in line.split("|")]
        rows.append(f)
    return rows


@pytest.mark.parametrize("row", _golden_rows(), ids=lambda r: f"{r[0]}-{r[8]}")
def test_storage_rate_matches_paper(row):
    name, H, I, E, d, K, r, bJ, quantity, printed, tol, _where = row
    bits = oracle.storage_bits_per_weight(int(d), int(K), int(r), int(H), int(I), int(E),
                                          b_J=int(bJ))
    value = bits if quantity == "bits" else 16.0 / bits
    assert abs(value - float(printed)) <= float(tol), (name, value)


def test_storage_rate_two_printed_forms_agree():
    # Section 5.5 prints 8/d + 16r/H + 16r/(EI) + 16Kd/(EHI) for K=256, 16-bit factors; the
    # appendix prints the general form.  They must be the same function.
    for (H, I, E, d, r) in [(2048, 768, 128, 8, 384), (2048, 1024, 64, 4, 256), (2816, 704, 128, 8, 512)]:
        K = 256
        sec55 = 8 / d + 16 * r / H + 16 * r / (E * I) + 16 * K * d / (E * H * I)
        assert abs(oracle.storage_bits_per_weight(d, K, r, H, I, E) - sec55) < 1e-12


def test_work_counts_and_read_reduction():
    # Appendix work table: HI/d selections and adds, Ir MACs, HK and Hr shared MACs.
    H, I, d, K, r = 2048, 768, 8, 256, 384
    wc = oracle.work_counts(H, I, d, K, r, b_J=8)
    assert wc["private_selections"] == H * I / d == wc["private_vq_adds"]
    assert wc["private_lowrank_macs"] == I * r
    assert wc["shared_codebook_macs"] == H * K and wc["shared_basis_macs"] == H * r
    # Section 5.2: MoE-projection HBM reads drop by 26-50 %; at Qwen3's deployed point with a
    # bf16 down projection the private bytes are exactly half of the dense expert's.
    private = 2 * (wc["private_index_bits"] + wc["private_coeff_bits"]) / 8 + 2 * H * I
    dense = 3 * 2 * H * I
    assert abs(1 - private / dense - 0.5) < 1e-12
    # Introduction: 75 MB of bf16 expert traffic per layer per token for Qwen3 (8 of 128 experts)
    assert abs(8 * dense / 1e6 - 75.5) < 0.1
    # Section 4.2: the two projection code books hold K*H/d bf16 values each: 0.25 MiB at d=8,
    # 0.5 MiB at d=4 (K=256, H=2048)
    assert 2 * (wc["shared_codebook_macs"] / d) * 2 / 2**20 == 0.25
    assert 2 * (oracle.work_counts(H, I, 4, K, r)["shared_codebook_macs"] / 4) * 2 / 2**20 == 0.5


# ------------------------------------------------------------------------------------------
# Eq. 1 by brute force in the paper's own orientation
# ------------------------------------------------------------------------------------------
def test_projection_matches_eq1_brute_force_in_paper_notation():
    shp = small_shape(H=24, I=10, E=3, K=7, r=3, T=1)
    layer = synth.make_layer(shp, seed=3)
    orc = oracle.OracleLayer.from_synth(layer)
    H, I, d, r = shp.H, shp.I, shp.d, shp.r
    h = f64(layer.x[0])
    for e in range(shp.E):
        # paper objects: code book (K x d), J_e (H/d x I), D (H x r), C_e (r x I)
        book = f64(layer.gate.codebook)
        J = layer.gate.idx[e].T.astype(int)
        D = f64(layer.gate.basis).T
        Ce = f64(layer.gate.factor[e]).T
        assert J.shape == (H // d, I) and D.shape == (H, r) and Ce.shape == (r, I)
        o = [0.0] * I
        for i in range(I):
            vq = 0.0
            for b in range(H // d):          # column i of Q(J_e): blocks stacked along H
                for j in range(d):
                    vq += book[J[b][i]][j] * h[b * d + j]
            z = [sum(D[m][rho] * h[m] for m in range(H)) for rho in range(r)]   # D^T h
            lr = sum(Ce[rho][i] * z[rho] for rho in range(r))                   # C_e^T z
            o[i] = vq + lr
        o = np.array(o)
        W = orc.reconstruct("gate", e)
        assert W.shape == (I, H)
        np.testing.assert_allclose(W @ h, o, rtol=0, atol=1e-13)
        np.testing.assert_allclose(orc.project_shared("gate", e, h), o, rtol=0, atol=1e-13)


def test_down_projection_blocks_run_along_intermediate_dim():
    shp = small_shape(H=16, I=40, E=2, K=9, r=2, T=1)
    layer = synth.make_layer(shp, seed=5)
    orc = oracle.OracleLayer.from_synth(layer)
    book = f64(layer.down.codebook)
    for e in range(shp.E):
        W = orc.reconstruct("down", e)
        assert W.shape == (shp.H, shp.I)
        lr = f64(layer.down.factor[e]) @ f64(layer.down.basis)
        for o_, b in itertools.product(range(shp.H), range(shp.I // shp.d)):
            blk = W[o_, b * shp.d:(b + 1) * shp.d] - lr[o_, b * shp.d:(b + 1) * shp.d]
            np.testing.assert_allclose(blk, book[layer.down.idx[e, o_, b]], atol=1e-15)


def test_vq_identity_projection_codebook_equals_reconstruction():
    shp = small_shape(H=64, I=16, K=32, r=5, T=1)
    layer = synth.make_layer(shp, seed=1)
    orc = oracle.OracleLayer.from_synth(layer)
    x = f64(layer.x[0])
    p = np.random.default_rng(0).standard_normal(shp.I)
    for e in range(shp.E):
        for proj, v in (("gate", x), ("up", x), ("down", p)):
            np.testing.assert_allclose(orc.project_shared(proj, e, v),
                                       orc.reconstruct(proj, e) @ v, rtol=0, atol=1e-12)


# ------------------------------------------------------------------------------------------
# special cases with closed forms
# ------------------------------------------------------------------------------------------
def test_all_indices_equal_gives_closed_form():
    shp = small_shape(r=0, T=1)
    layer = synth.make_layer(shp, seed=2)
    layer.gate.idx[:] = 5
    orc = oracle.OracleLayer.from_synth(layer)
    x = f64(layer.x[0])
    c = f64(layer.gate.codebook[5])
    closed = sum(float(c @ x[b * shp.d:(b + 1) * shp.d]) for b in range(shp.H // shp.d))
    np.testing.assert_allclose(orc.reconstruct("gate", 0) @ x, np.full(shp.I, closed), atol=1e-13)


def test_zero_codebook_is_pure_low_rank_layer():
    shp = small_shape(K=1, r=6, T=2)
    layer = synth.make_layer(shp, seed=4)
    for p in (layer.gate, layer.up, layer.down):
        p.codebook[:] = 0
    orc = oracle.OracleLayer.from_synth(layer)
    for e in range(shp.E):
        AB = f64(layer.up.factor[e]) @ f64(layer.up.basis)      # (A_e B) materialised
        np.testing.assert_allclose(orc.reconstruct("up", e), AB, atol=1e-15)
        x = f64(layer.x[1])
        np.testing.assert_allclose(orc.reconstruct("up", e) @ x,
                                   f64(layer.up.factor[e]) @ (f64(layer.up.basis) @ x),
                                   atol=1e-13)


def _dense_from_blocks(layer, proj):
    """Dense bf16 matrices whose every length-d block is literally a code word."""
    P = getattr(layer, proj)
    n_exp, out_dim, nb = P.idx.shape
    return P.codebook[P.idx.astype(np.int64)].reshape(n_exp, out_dim, nb * P.codebook.shape[1])


def _torch_mlp(Wg, Wu, Wd, x):
    g = torch.nn.functional.linear(x, Wg)
    u = torch.nn.functional.linear(x, Wu)
    return torch.nn.functional.linear(torch.nn.functional.silu(g) * u, Wd)


def test_exact_codebook_rank0_reproduces_dense_bf16_expert():
    shp = small_shape(r=0, T=3, k=2)
    layer = synth.make_layer(shp, seed=7)
    comp = oracle.OracleLayer.from_synth(layer).decode_layer(layer.x)
    dense_layer = synth.make_layer(synth.replace(shp, mode="dense"), seed=7)
    dense_layer.router_w, dense_layer.x = layer.router_w, layer.x
    for proj in ("gate", "up", "down"):
        getattr(dense_layer, proj).dense = _dense_from_blocks(layer, proj)
    dense = oracle.OracleLayer.from_synth(dense_layer).decode_layer(layer.x)
    np.testing.assert_array_equal(comp.topk_id, dense.topk_id)
    np.testing.assert_allclose(comp.out, dense.out, rtol=0, atol=1e-12)
    # and against a library MLP on the dense matrices, expert by expert
    xt = torch.from_numpy(f64(layer.x))
    for t in range(shp.T):
        acc = torch.zeros(shp.H, dtype=torch.float64)
        for s in range(shp.k):
            e = int(comp.topk_id[t, s])
            Wg, Wu, Wd = (torch.from_numpy(f64(getattr(dense_layer, p).dense[e]))
                          for p in ("gate", "up", "down"))
            acc += comp.topk_w[t, s] * _torch_mlp(Wg, Wu, Wd, xt[t])
        np.testing.assert_allclose(comp.out[t], acc.numpy(), rtol=0, atol=1e-12)


@pytest.mark.parametrize("d", [8, 4, 2])
def test_single_expert_is_plain_swiglu_mlp(d):
    shp = small_shape(E=1, k=1, T=2, r=3, d=d)
    layer = synth.make_layer(shp, seed=8)
    orc = oracle.OracleLayer.from_synth(layer)
    res = orc.decode_layer(layer.x)
    assert np.all(res.topk_id == 0) and np.allclose(res.topk_w, 1.0)
    W = {}
    for p in ("gate", "up", "down"):
        P = getattr(layer, p)
        W[p] = torch.from_numpy(f64(P.codebook)[P.idx[0].astype(int)].reshape(P.out_dim, P.in_dim)
                                + f64(P.factor[0]) @ f64(P.basis))
    ref = _torch_mlp(W["gate"], W["up"], W["down"], torch.from_numpy(f64(layer.x)))
    np.testing.assert_allclose(res.out, ref.numpy(), rtol=0, atol=1e-12)


def test_storage_rate_sweep_shapes_hit_their_rates():
    # Section 5.5: K = 256, d in {8, 4}, r chosen for about 3, 4 and 5 bits per original weight
    # (here r is a multiple of 8, which moves the 3-bit point 0.022 off its target)
    for name, target in (("qwen3_3bit", 3.0), ("qwen3_4bit", 4.0), ("qwen3_5bit", 5.0),
                         ("qwen3_d4_3bit", 3.0), ("qwen3_d4_4bit", 4.0), ("qwen3_d4_5bit", 5.0)):
        s = synth.shape(name)
        bits = oracle.storage_bits_per_weight(s.d, s.K, s.r, s.H, s.I, s.E)
        closed = 8 / s.d + 16 * s.r / s.H + 16 * s.r / (s.E * s.I) + 16 * s.K * s.d / (s.E * s.H * s.I)
        assert abs(bits - closed) < 1e-12
        assert abs(bits - target) < 0.025, (name, bits)


def test_activations_match_library_and_closed_forms():
    # Section 2.1 leaves the expert activation to the model: SiLU and the tanh form of GELU
    v = np.concatenate([np.linspace(-12, 12, 97), [0.0, 1e-9, -1e-9, 30.0, -30.0]])
    tv = torch.from_numpy(v)
    np.testing.assert_allclose(oracle.activation(v, "silu"), torch.nn.functional.silu(tv).numpy(),
                               rtol=0, atol=1e-14)
    np.testing.assert_allclose(oracle.activation(v, "gelu_tanh"),
                               torch.nn.functional.gelu(tv, approximate="tanh").numpy(), rtol=0, atol=1e-14)
    for act in ("silu", "gelu_tanh"):
        a = oracle.activation(v, act)
        np.testing.assert_allclose(a - oracle.activation(-v, act), v, rtol=0, atol=1e-13)   # phi(v) - phi(-v) = v
        assert oracle.activation(0.0, act)[0] == 0.0
        assert abs(oracle.activation(30.0, act)[0] - 30.0) < 1e-9 and abs(oracle.activation(-30.0, act)[0]) < 1e-9
    # the two differ where it matters (a flag that is ignored must not pass a parity test)
    assert abs(oracle.activation(1.0, "silu")[0] - 0.7310585786300049) < 1e-15
    assert abs(oracle.activation(1.0, "gelu_tanh")[0] - 0.8411919906082768) < 1e-13
    # against the exact GELU v * Phi(v) the tanh form stays within its known 5e-4 error
    exact = v * 0.5 * (1.0 + torch.erf(tv / np.sqrt(2.0)).numpy())
    assert np.max(np.abs(oracle.activation(v, "gelu_tanh") - exact)) < 5e-4


def test_single_expert_with_gelu_is_plain_geglu_mlp():
    shp = small_shape(E=1, k=1, T=2, r=3, act="gelu_tanh")
    layer = synth.make_layer(shp, seed=8)
    res = oracle.OracleLayer.from_synth(layer).decode_layer(layer.x)
    W = {}
    for p in ("gate", "up", "down"):
        P = getattr(layer, p)
        W[p] = torch.from_numpy(f64(P.codebook)[P.idx[0].astype(int)].reshape(P.out_dim, P.in_dim)
                                + f64(P.factor[0]) @ f64(P.basis))
    xt = torch.from_numpy(f64(layer.x))
    lin = torch.nn.functional.linear
    ref = lin(torch.nn.functional.gelu(lin(xt, W["gate"]), approximate="tanh") * lin(xt, W["up"]), W["down"])
    np.testing.assert_allclose(res.out, ref.numpy(), rtol=0, atol=1e-12)
    silu = oracle.OracleLayer.from_synth(layer, act="silu").decode_layer(layer.x)
    assert np.max(np.abs(silu.out - res.out)) > 1e-3 * np.max(np.abs(res.out))


# ------------------------------------------------------------------------------------------
# router, affinities, grouping, combine
# ------------------------------------------------------------------------------------------
def test_router_logits_match_library_matmul():
    shp = small_shape(T=4, router_bias=True)
    layer = synth.make_layer(shp, seed=9)
    res = oracle.OracleLayer.from_synth(layer).decode_layer(layer.x)
    ref = f64(layer.x) @ f64(layer.router_w).T + layer.router_bias.astype(np.float64)
    np.testing.assert_allclose(res.logits, ref, rtol=0, atol=1e-13)


def test_affinities_sum_to_one_and_order():
    shp = small_shape(E=16, k=5, T=7, router_bias=True)
    layer = synth.make_layer(shp, seed=10)
    res = oracle.OracleLayer.from_synth(layer).decode_layer(layer.x)
    np.testing.assert_allclose(res.topk_w.sum(axis=1), 1.0, rtol=0, atol=1e-15)
    for t in range(shp.T):
        order = sorted(range(shp.E), key=lambda e: (-res.logits[t, e], e))[:shp.k]
        assert list(res.topk_id[t]) == order
        sel = res.logits[t, order]
        np.testing.assert_allclose(res.topk_w[t], torch.softmax(torch.from_numpy(sel), 0).numpy(),
                                   atol=1e-15)


def test_no_renorm_is_softmax_over_all_experts():
    logits = np.random.default_rng(0).standard_normal((3, 9))
    ids, w = oracle.topk_affinity(logits, 4, renorm=False)
    full = torch.softmax(torch.from_numpy(logits), dim=1).numpy()
    for t in range(3):
        np.testing.assert_allclose(w[t], full[t, ids[t]], atol=1e-15)


def test_exact_ties_go_to_lower_expert_id():
    logits = np.array([[0.5, 2.0, 2.0, -1.0, 2.0, 0.5]])
    ids, w = oracle.topk_affinity(logits, 4)
    assert ids.tolist() == [[1, 2, 4, 0]]
    # through the layer: duplicated router rows tie exactly
    shp = small_shape(E=8, k=3, T=5)
    layer = synth.make_layer(shp, seed=11)
    synth.duplicate_router_rows(layer, src=6, dst=2)
    res = oracle.OracleLayer.from_synth(layer).decode_layer(layer.x)
    assert np.array_equal(res.logits[:, 6], res.logits[:, 2])
    for t in range(shp.T):
        row = list(res.topk_id[t])
        if 6 in row:
            assert 2 in row and row.index(2) == row.index(6) - 1


def test_topk_equal_E_is_dense_mixture():
    shp = small_shape(E=5, k=5, T=3, r=3)
    layer = synth.make_layer(shp, seed=12)
    orc = oracle.OracleLayer.from_synth(layer)
    res = orc.decode_layer(layer.x)
    x = f64(layer.x)
    logits = x @ f64(layer.router_w).T
    a = torch.softmax(torch.from_numpy(logits), dim=1).numpy()
    ref = np.zeros((shp.T, shp.H))
    for e in range(shp.E):
        Wg, Wu, Wd = (orc.reconstruct(p, e) for p in ("gate", "up", "down"))
        g, u = x @ Wg.T, x @ Wu.T
        ref += a[:, e:e + 1] * ((g / (1 + np.exp(-g)) * u) @ Wd.T)
    np.testing.assert_allclose(res.out, ref, rtol=0, atol=1e-12)


def test_permuting_experts_permutes_ids_and_keeps_output():
    shp = small_shape(E=6, k=2, T=4, mode="paper")
    layer = synth.make_layer(shp, seed=13)
    res = oracle.OracleLayer.from_synth(layer).decode_layer(layer.x)
    perm = np.random.default_rng(1).permutation(shp.E)          # new id j holds old expert perm[j]
    inv = np.argsort(perm)
    layer2 = synth.make_layer(shp, seed=13)
    layer2.router_w = layer.router_w[perm]
    for p in ("gate", "up", "down"):
        P, P2 = getattr(layer, p), getattr(layer2, p)
        for f in ("idx", "factor", "dense"):
            if getattr(P, f) is not None:
                setattr(P2, f, getattr(P, f)[perm])
    res2 = oracle.OracleLayer.from_synth(layer2).decode_layer(layer.x)
    np.testing.assert_array_equal(res2.topk_id, inv[res.topk_id])
    np.testing.assert_allclose(res2.out, res.out, rtol=0, atol=1e-13)


def test_grouping_brute_force():
    rng = np.random.default_rng(2)
    for T, k, E in [(1, 2, 8), (4, 3, 5), (16, 8, 128), (3, 1, 2)]:
        ids = np.stack([rng.permutation(E)[:k] for _ in range(T)]).astype(np.int32)
        counts, offsets, ptok, pslot = oracle.group_by_expert(ids, E)
        assert counts.sum() == T * k and offsets[0] == 0 and offsets[-1] == T * k
        assert np.array_equal(np.diff(offsets), counts)
        assert np.array_equal(counts, np.bincount(ids.ravel(), minlength=E))
        seen = set()
        for e in range(E):
            toks = ptok[offsets[e]:offsets[e + 1]]
            assert np.all(np.diff(toks) > 0)                   # ascending tokens, no repeats
            for q in range(offsets[e], offsets[e + 1]):
                assert ids[ptok[q], pslot[q]] == e
                seen.add((int(ptok[q]), int(pslot[q])))
        assert len(seen) == T * k


def test_shared_experts_enter_with_weight_one():
    shp = small_shape(E=4, k=2, S=2, T=2)
    layer = synth.make_layer(shp, seed=14)
    orc = oracle.OracleLayer.from_synth(layer)
    res = orc.decode_layer(layer.x)
    x = f64(layer.x)
    for t in range(shp.T):
        acc = np.zeros(shp.H)
        for s in range(shp.k + shp.S):
            e = int(res.topk_id[t, s]) if s < shp.k else shp.E + (s - shp.k)
            a = res.topk_w[t, s] if s < shp.k else 1.0
            Wg, Wu, Wd = (orc.reconstruct(p, e) for p in ("gate", "up", "down"))
            g, u = Wg @ x[t], Wu @ x[t]
            y = Wd @ (g / (1 + np.exp(-g)) * u)
            np.testing.assert_allclose(res.y_pair[t, s], y, atol=1e-13)
            acc += a * y
        np.testing.assert_allclose(res.out[t], acc, atol=1e-13)


def test_sampled_down_rows_equal_full_result():
    shp = small_shape(T=2, mode="paper")
    layer = synth.make_layer(shp, seed=15)
    orc = oracle.OracleLayer.from_synth(layer)
    full = orc.decode_layer(layer.x)
    rows = [0, 7, 13, shp.H - 1]
    part = orc.decode_layer(layer.x, down_rows=rows)
    np.testing.assert_array_equal(part.out, full.out[:, rows])


def test_bad_index_is_reported():
    shp = small_shape(K=5, T=1)
    layer = synth.make_layer(shp, seed=16)
    res0 = oracle.OracleLayer.from_synth(layer).decode_layer(layer.x)
    assert not res0.bad_index
    e = int(res0.topk_id[0, 0])
    layer.up.idx[e, 3, 1] = 5
    assert oracle.OracleLayer.from_synth(layer).decode_layer(layer.x).bad_index


def test_generator_is_deterministic_and_bf16_exact():
    a = synth.make_layer(synth.shape("tiny"), seed=0)
    b = synth.make_layer(synth.shape("tiny"), seed=0)
    assert np.array_equal(a.gate.idx, b.gate.idx) and np.array_equal(a.x, b.x)
    assert a.gate.codebook is a.up.codebook is a.down.codebook
    v = np.array([1.0, 1.00390625, 1.005859375, -2.5, 3.0e-5], np.float32)
    bits = synth.f32_to_bf16_bits(v)
    ref = torch.from_numpy(v).to(torch.bfloat16).view(torch.int16).numpy().view(np.uint16)
    assert np.array_equal(bits, ref)


# ------------------------------------------------------------------------------------------
# up-only ReLU^2 experts (Section 5.7: the Nemotron-shaped layer) and a padded hidden dimension
# ------------------------------------------------------------------------------------------
def test_single_up_only_expert_is_plain_relu2_mlp():
    """E = 1, k = 1, no gate projection: the layer is x -> W_down relu(W_up x)^2, computed here by
    torch in fp64 from the oracle's own reconstruction of the two matrices."""
    shp = small_shape(E=1, k=1, T=3, r=3, act="relu2")
    layer = synth.make_layer(shp, 9)
    assert layer.gate is None
    orc = oracle.OracleLayer.from_synth(layer)
    res = orc.decode_layer(layer.x)
    W = {}
    for p in ("up", "down"):                       # Eq. 1 written out with numpy, not the oracle's routine
        P = getattr(layer, p)
        W[p] = torch.from_numpy(f64(P.codebook)[P.idx[0].astype(int)].reshape(P.out_dim, P.in_dim)
                                + f64(P.factor[0]) @ f64(P.basis))
    Wu, Wd = W["up"], W["down"]
    xt = torch.from_numpy(f64(layer.x))
    ref = (torch.relu(xt @ Wu.T) ** 2) @ Wd.T
    np.testing.assert_allclose(res.out, ref.numpy(), rtol=1e-12, atol=1e-14)
    # p >= 0 everywhere, so flipping the sign of the tokens changes the result unless u == 0
    neg = layer.x ^ np.uint16(0x8000)
    res2 = orc.decode_layer(neg)
    ref2 = (torch.relu(-xt @ Wu.T) ** 2) @ Wd.T
    np.testing.assert_allclose(res2.out, ref2.numpy(), rtol=1e-12, atol=1e-14)
    assert np.max(np.abs(res2.out - res.out)) > 1e-6


def test_up_only_differs_from_a_gated_expert_and_ignores_a_gate():
    shp = small_shape(T=2, act="relu2")
    up_only = synth.make_layer(shp, 4)
    res = oracle.OracleLayer.from_synth(up_only).decode_layer(up_only.x)
    # the same layer with SOME gate attached and the up-only activation: the gate must not be read
    gated = synth.make_layer(small_shape(T=2), 5)
    mixed = synth.Layer(shape=shp, router_w=up_only.router_w, router_bias=None, x=up_only.x, gate=gated.gate,
                        up=up_only.up, down=up_only.down)
    res_mixed = oracle.OracleLayer.from_synth(mixed, act="relu2").decode_layer(up_only.x)
    np.testing.assert_array_equal(res_mixed.out, res.out)
    res_silu = oracle.OracleLayer.from_synth(mixed, act="silu").decode_layer(up_only.x)
    assert np.max(np.abs(res_silu.out - res.out)) > 1e-3 * np.max(np.abs(res.out))


def test_padding_the_hidden_dimension_with_zero_activations_changes_nothing():
    """A hidden size that is not a multiple of the block length is padded (Section 5.7): the
    padded tokens carry zeros there, so whatever the padded weight columns hold -- here random
    code words and a random low-rank part -- the output rows of the true hidden size equal a dense
    evaluation on the unpadded matrices."""
    H_true, H_pad = 44, 48
    shp = small_shape(H=H_pad, E=1, k=1, T=2, act="relu2")
    layer = synth.make_layer(shp, 11)
    x = layer.x.copy()
    x[:, H_true:] = 0                              # bf16 +0
    orc = oracle.OracleLayer.from_synth(layer)
    res = orc.decode_layer(x)
    Wu = torch.from_numpy(orc.reconstruct("up", 0))[:, :H_true]           # I x H_true
    Wd = torch.from_numpy(orc.reconstruct("down", 0))[:H_true]            # H_true x I
    xt = torch.from_numpy(f64(x))[:, :H_true]
    ref = (torch.relu(xt @ Wu.T) ** 2) @ Wd.T
    np.testing.assert_allclose(res.out[:, :H_true], ref.numpy(), rtol=1e-12, atol=1e-14)


# ------------------------------------------------------------------------------------------
# twelve-bit packed indices (Appendix "Exact engine-work counts": the index width b_J(K))
# ------------------------------------------------------------------------------------------
def test_packed_twelve_bit_indices_round_trip_and_equal_the_uint16_layer():
    rng = np.random.default_rng(0)
    idx = rng.integers(0, 4096, size=(3, 5, 16), dtype=np.uint16)
    idx[0, 0, :4] = [0, 4095, 0x0F0, 0xA05]        # extremes and both nibble positions
    packed = synth.pack12(idx)
    assert packed.dtype == np.uint8 and packed.shape == (3, 5, 24)
    # bytes of the first pair by hand: 0x000, 0xFFF -> 00 F0 FF
    assert packed[0, 0, :3].tolist() == [0x00, 0xF0, 0xFF]
    flat = idx.reshape(-1)
    for pos in list(range(40)) + [flat.size - 1]:
        assert oracle.read_index(packed, 12, pos) == int(flat[pos])
    # storage: twelve bits per index is three quarters of the uint16 map
    assert packed.nbytes * 4 == idx.nbytes * 3
    assert abs(oracle.storage_bits_per_weight(8, 4096, 0, 2048, 768, 128, b_J=12)
               - (12 / 8 + 16 * 4096 * 8 / (128 * 2048 * 768))) < 1e-12
    # the layer: same draws, indices packed -> bit-identical oracle output, on every projection
    a = synth.make_layer(small_shape(K=700, T=2, I=32), 3)           # rows of 6 (gate, up) and 4 (down) indices
    b = synth.make_layer(small_shape(K=700, T=2, I=32, idx12=True), 3)
    assert b.gate.idx.dtype == np.uint8 and b.gate.idx_bits == 12
    ra = oracle.OracleLayer.from_synth(a).decode_layer(a.x)
    rb = oracle.OracleLayer.from_synth(b).decode_layer(b.x)
    np.testing.assert_array_equal(ra.out, rb.out)
    np.testing.assert_array_equal(oracle.OracleLayer.from_synth(b).reconstruct("down", 2),
                                  oracle.OracleLayer.from_synth(a).reconstruct("down", 2))
