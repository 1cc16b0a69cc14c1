"""Pins of the oracle's node-subset layer (Algorithm 1, Stage 2: the correction tokens are re-forwarded through the
shallow layers under tree-masked attention while the main-chain nodes already sit in the KV cache).

What fixes the expected values: torch's scaled_dot_product_attention with an explicit boolean mask, and the whole-tree
layer (itself pinned against HuggingFace LLaMA): a node's output depends only on its own hidden state and on the K/V
rows of the prefix and of its ancestors, so forwarding the chain first and the corrections afterwards must reproduce
the one-shot forward of the whole tree bit for bit."""
import numpy as np
import pytest
import torch

import oracle
from paper_2605_11186_b200 import inputs as gen
from helpers import ref_cfg, np_model


@pytest.fixture(autouse=True)
def _contract_on():
    oracle.set_contract(True)
    yield
    oracle.set_contract(True)


def _bits(mask_row, T):
    return np.array([(int(mask_row[j >> 6]) >> (j & 63)) & 1 for j in range(T)], bool)


def test_subset_attention_matches_torch_sdpa():
    oracle.set_contract(False)
    rng = np.random.default_rng(11)
    parent = gen.tree_random(70, 5)
    T, P, nh, hd = 70, 21, 3, 16
    _, mask, _, _ = oracle.build_tree_mask(parent, P)
    rows = np.array([3, 17, 40, 64, 69], np.int32)       # crosses the 64-bit word boundary
    q = rng.standard_normal((len(rows), nh, hd))
    kc = rng.standard_normal((P + T, nh * hd)).astype(np.float32)
    vc = rng.standard_normal((P + T, nh * hd)).astype(np.float32)
    got = oracle.tree_attention_rows(q, kc, vc, mask[rows], T, P, nh, hd, 0.3)
    bm = np.ones((len(rows), P + T), bool)
    for j, n in enumerate(rows):
        bm[j, P:] = _bits(mask[n], T)
    tq = torch.from_numpy(q).permute(1, 0, 2)[None]
    tk = torch.from_numpy(kc.astype(np.float64)).view(P + T, nh, hd).permute(1, 0, 2)[None]
    tv = torch.from_numpy(vc.astype(np.float64)).view(P + T, nh, hd).permute(1, 0, 2)[None]
    want = torch.nn.functional.scaled_dot_product_attention(tq, tk, tv, attn_mask=torch.from_numpy(bm)[None, None], scale=0.3)
    assert np.abs(got - want[0].permute(1, 0, 2).numpy()).max() < 1e-12
    # the same rows through the whole-tree routine
    q_all = rng.standard_normal((T, nh, hd))
    q_all[rows] = q
    full = oracle.tree_attention(q_all, kc, vc, mask, P, nh, hd, 0.3)
    assert np.array_equal(full[rows], got)


@pytest.fixture(scope="module")
def ctx():
    m = gen.TINY
    model = gen.make_model(m, "subset")
    nm = np_model(model)
    P, max_seq = 40, 200
    cfg = ref_cfg(m, max_seq)
    D = m.n_heads * m.head_dim
    kc = oracle.from_bf16(gen.bf16_bits(gen.normal_bf16((m.n_layers, max_seq, D), 1.0, "cpu", "subset", "k"))).copy()
    vc = oracle.from_bf16(gen.bf16_bits(gen.normal_bf16((m.n_layers, max_seq, D), 1.0, "cpu", "subset", "v"))).copy()
    return dict(m=m, nm=nm, cfg=cfg, P=P, kc=kc, vc=vc)


def _full(ctx, parent, tokens):
    """All layers over the whole tree, layer by layer: (resid after every layer, caches)."""
    m, nm, cfg, P = ctx["m"], ctx["nm"], ctx["cfg"], ctx["P"]
    kc, vc = ctx["kc"].copy(), ctx["vc"].copy()
    _, mask, pos, _ = oracle.build_tree_mask(parent, P)
    resid = oracle.embed(nm["embed"], tokens)
    per_layer = []
    for l in range(m.n_layers):
        oracle.verify_layer(cfg, nm["layers"][l], resid, kc[l], vc[l], mask, pos, P)
        per_layer.append(resid.copy())
    return per_layer, kc, vc, mask, pos


@pytest.mark.parametrize("gamma,corr", [(5, [1, 3]), (7, [0]), (5, [0, 1, 2, 3, 4]), (3, [2])])
def test_reforward_of_corrections_equals_one_shot_tree_forward(ctx, gamma, corr):
    m, nm, cfg, P = ctx["m"], ctx["nm"], ctx["cfg"], ctx["P"]
    parent = gen.tree_cats(gamma, corr)
    T = len(parent)
    tokens = gen.uniform_tokens(T, m.vocab, "subset", gamma)
    per_layer, kc_full, vc_full, mask, pos = _full(ctx, parent, tokens)

    # Stage 1/2 order: the main chain (nodes 0..gamma) first ...
    kc, vc = ctx["kc"].copy(), ctx["vc"].copy()
    chain = np.arange(gamma + 1, dtype=np.int32)
    resid_c = oracle.embed(nm["embed"], tokens[chain])
    for l in range(m.n_layers):
        assert oracle.verify_layer_nodes(cfg, nm["layers"][l], resid_c, kc[l], vc[l], mask, pos, chain, P) == 0
        assert np.array_equal(resid_c, per_layer[l][chain])
    # ... then only the correction nodes, against the chain's cached rows
    nodes = np.arange(gamma + 1, T, dtype=np.int32)
    before_k = kc.copy()
    resid_s = oracle.embed(nm["embed"], tokens[nodes])
    for l in range(m.n_layers):
        assert oracle.verify_layer_nodes(cfg, nm["layers"][l], resid_s, kc[l], vc[l], mask, pos, nodes, P) == 0
        assert np.array_equal(resid_s, per_layer[l][nodes]), "layer %d" % l
    assert np.array_equal(kc, kc_full) and np.array_equal(vc, vc_full)
    keep = np.ones(kc.shape[1], bool)
    keep[P + nodes] = False
    assert np.array_equal(kc[:, keep], before_k[:, keep])       # only the active nodes' rows were written


def test_subset_with_active_ancestors_and_all_nodes(ctx):
    """A whole subtree re-forwarded at once (active nodes that are ancestors of active nodes), and nodes = all."""
    m, nm, cfg, P = ctx["m"], ctx["nm"], ctx["cfg"], ctx["P"]
    parent = gen.tree_random(37, 7)
    T = len(parent)
    tokens = gen.uniform_tokens(T, m.vocab, "subset", "rand")
    per_layer, kc_full, vc_full, mask, pos = _full(ctx, parent, tokens)
    # subtree of node 2, plus everything outside it already cached
    sub = [i for i in range(T) if (int(mask[i][0]) >> 2) & 1]
    assert len(sub) >= 3 and len(sub) < T
    nodes = np.asarray(sub, np.int32)
    kc, vc = kc_full.copy(), vc_full.copy()
    kc[:, P + nodes] = np.nan                                    # the active rows must come from this call
    vc[:, P + nodes] = np.nan
    resid = oracle.embed(nm["embed"], tokens[nodes])
    for l in range(m.n_layers):
        assert oracle.verify_layer_nodes(cfg, nm["layers"][l], resid, kc[l], vc[l], mask, pos, nodes, P) == 0
        assert np.array_equal(resid, per_layer[l][nodes])
    assert np.array_equal(kc, kc_full) and np.array_equal(vc, vc_full)

    kc, vc = ctx["kc"].copy(), ctx["vc"].copy()
    resid = oracle.embed(nm["embed"], tokens)
    every = np.arange(T, dtype=np.int32)
    for l in range(m.n_layers):
        oracle.verify_layer_nodes(cfg, nm["layers"][l], resid, kc[l], vc[l], mask, pos, every, P)
        assert np.array_equal(resid, per_layer[l])


def test_subset_rejects_bad_node_lists(ctx):
    m, nm, cfg, P = ctx["m"], ctx["nm"], ctx["cfg"], ctx["P"]
    parent = gen.tree_cats(4, [1])
    _, mask, pos, _ = oracle.build_tree_mask(parent, P)
    kc, vc = ctx["kc"][0].copy(), ctx["vc"][0].copy()
    for bad in ([3, 2], [2, 2], [-1, 2], [2, 6]):
        resid = np.zeros((2, m.hidden), np.float32)
        assert oracle.verify_layer_nodes(cfg, nm["layers"][0], resid, kc, vc, mask, pos, np.asarray(bad, np.int32), P) != 0
