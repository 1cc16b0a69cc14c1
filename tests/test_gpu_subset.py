"""GPU parity of the partial-tree layer (Algorithm 1, Stage 2: correction tokens re-forwarded under tree-masked attention
against the main chain's cached K/V): cats_verify_layer_nodes against the oracle's verify_layer_nodes on the same seeded
inputs, in the order the algorithm runs them (chain first, corrections afterwards), and against the one-shot layer over
the whole tree on the GPU."""
import numpy as np
import pytest
import torch

import oracle
from paper_2605_11186_b200 import inputs as gen
from helpers import ref_cfg, np_layer, cache_to_f32
from test_gpu_parity import TOL, dev, dev_layer, contract_floor, bf16_ulp_close

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def cats():
    from paper_2605_11186_b200 import binding
    assert torch.cuda.is_available()
    return binding


def _case(cats, m, tag, parent, nodes_first, nodes_second, P, resid_std):
    """Forward nodes_first, then nodes_second (both ascending lists of tree nodes), one layer; compare both steps."""
    T = len(parent)
    max_seq = P + T
    w = gen.make_layer(m, tag, 0)
    kc, vc = gen.make_kv_prefix(m, 1, max_seq, P, tag)
    resid = (gen.normal_bf16((T, m.hidden), resid_std, "cpu", tag, "resid").float()
             + 1e-3 * gen.normal_bf16((T, m.hidden), 1.0, "cpu", tag, "resid_lo").float())
    _, mask, pos, _ = oracle.build_tree_mask(parent, P)
    rcfg = ref_cfg(m, max_seq, 1)
    nw = np_layer(w)
    steps = [np.asarray(n, np.int32) for n in (nodes_first, nodes_second) if len(n)]

    def run():
        r_k, r_v = cache_to_f32(kc[0]), cache_to_f32(vc[0])
        outs = []
        for nodes in steps:
            r = resid.numpy()[nodes].copy()
            assert oracle.verify_layer_nodes(rcfg, nw, r, r_k, r_v, mask, pos, nodes, P) == 0
            outs.append(r)
        return outs + [r_k, r_v]
    ref, floor = contract_floor(run)
    r_k, r_v = ref[-2], ref[-1]

    cfg = cats.model_cfg(m, max_seq, 1)
    dw = cats.pack_layer(dev_layer(w))
    lw = cats.layer_weights(dw)
    d_k, d_v = kc[0].cuda(), vc[0].cuda()
    ws = cats.new_workspace(cfg, T, P)
    d_mask, d_pos = dev(mask.view(np.int64)), dev(pos)
    got = []
    for nodes in steps:
        st = cats.new_status()
        d_resid = resid[torch.from_numpy(nodes).long()].contiguous().cuda()
        cats.cats_verify_layer_nodes(cfg, lw, d_resid, d_k, d_v, d_mask, d_pos, dev(nodes), T, P, ws, st)
        torch.cuda.synchronize()
        assert int(st.item()) == 0
        got.append(d_resid.cpu().numpy())
    for i, (g, r) in enumerate(zip(got, ref)):
        tol = max(TOL, 3.0 * floor[i])
        err = np.abs(g - r).max()
        assert err <= tol, (i, err, tol)
    written = np.concatenate(steps)
    for d, r, orig in ((d_k, r_k, kc), (d_v, r_v, vc)):
        nbad, maxerr = bf16_ulp_close(d[torch.from_numpy(P + written).long().cuda()], r[P + written])
        assert nbad == 0, (nbad, maxerr)
        untouched = np.ones(max_seq, bool)
        untouched[P + written] = False
        idx = torch.from_numpy(np.nonzero(untouched)[0])
        assert torch.equal(d.cpu()[idx], orig[0][idx])
    return got, steps, (w, kc, vc, resid, mask, pos, cfg, lw, dw)


CATS_TREES = [
    ("g5_c13", 5, [1, 3]), ("g7_c0", 7, [0]), ("g5_all", 5, [0, 1, 2, 3, 4]), ("g10_c259", 10, [2, 5, 9]),
]


@pytest.mark.parametrize("name,gamma,corr", CATS_TREES, ids=[c[0] for c in CATS_TREES])
def test_stage2_order_tiny(cats, name, gamma, corr):
    parent = gen.tree_cats(gamma, corr)
    chain = list(range(gamma + 1))
    _case(cats, gen.TINY, ("subset_tiny", name), parent, chain, list(range(gamma + 1, len(parent))), 77, 1.0)


def test_stage2_order_7b_shape_and_one_shot_equivalence(cats):
    """7B-shaped layer, prefix 512, gamma = 5 with three corrections; the two-step result must also agree with the one-shot
    layer over the whole tree on the GPU (same K/V rows bit for bit: they do not depend on which rows share a launch)."""
    gamma, corr = 5, [0, 2, 4]
    parent = gen.tree_cats(gamma, corr)
    T, P = len(parent), 512
    m = gen.LLAMA_7B
    got, steps, (w, kc, vc, resid, mask, pos, cfg, lw, dw) = _case(
        cats, m, "subset_7b", parent, list(range(gamma + 1)), list(range(gamma + 1, T)), P, 1.0)
    d_k, d_v = kc[0].cuda(), vc[0].cuda()
    d_resid = resid.cuda()
    ws = cats.new_workspace(cfg, T, P)
    st = cats.new_status()
    cats.cats_verify_layer(cfg, lw, d_resid, d_k, d_v, dev(mask.view(np.int64)), dev(pos), T, P, ws, st)
    torch.cuda.synchronize()
    assert int(st.item()) == 0
    full = d_resid.cpu().numpy()
    two_step = np.concatenate(got)
    assert np.abs(full - two_step).max() <= TOL


def test_subtree_and_scattered_nodes_tiny(cats):
    """Active nodes that are ancestors of other active nodes; a scattered list crossing the 64-node word boundary."""
    parent = gen.tree_random(100, 3)
    _, mask, _, _ = oracle.build_tree_mask(parent, 0)
    sub = [i for i in range(100) if (int(mask[i][0]) >> 1) & 1]          # subtree of node 1
    rest = [i for i in range(100) if i not in sub]
    assert len(sub) >= 3
    _case(cats, gen.TINY, "subset_subtree", parent, rest, sub, 33, 1.0)


def test_all_nodes_equals_whole_tree_layer(cats):
    parent = gen.tree_branching([4, 2, 1, 1], 16)
    T, P, m = 16, 128, gen.TINY
    got, steps, (w, kc, vc, resid, mask, pos, cfg, lw, dw) = _case(cats, m, "subset_all", parent, list(range(T)), [], P, 1.0)
    d_k, d_v, d_resid = kc[0].cuda(), vc[0].cuda(), resid.cuda()
    ws = cats.new_workspace(cfg, T, P)
    st = cats.new_status()
    cats.cats_verify_layer(cfg, lw, d_resid, d_k, d_v, dev(mask.view(np.int64)), dev(pos), T, P, ws, st)
    torch.cuda.synchronize()
    assert np.array_equal(d_resid.cpu().numpy(), got[0])                 # same kernels, same launch shapes


def test_malformed_node_list_is_reported_not_followed(cats):
    parent = gen.tree_cats(4, [1])
    T, P, m = len(parent), 16, gen.TINY
    max_seq = P + T
    w = gen.make_layer(m, "subset_bad", 0)
    kc, vc = gen.make_kv_prefix(m, 1, max_seq, P, "subset_bad")
    _, mask, pos, _ = oracle.build_tree_mask(parent, P)
    cfg = cats.model_cfg(m, max_seq, 1)
    dw = cats.pack_layer(dev_layer(w))
    ws = cats.new_workspace(cfg, T, P)
    for bad in ([3, 2], [2, 2], [-5, 2], [2, 4000]):
        st = cats.new_status()
        d_k, d_v = kc[0].cuda(), vc[0].cuda()
        d_resid = torch.zeros((2, m.hidden), dtype=torch.float32, device="cuda")
        cats.cats_verify_layer_nodes(cfg, cats.layer_weights(dw), d_resid, d_k, d_v, dev(mask.view(np.int64)), dev(pos),
                                     dev(np.asarray(bad, np.int32)), T, P, ws, st)
        torch.cuda.synchronize()
        assert int(st.item()) == -1
        assert torch.equal(d_k[:P].cpu(), kc[0, :P])                     # the prefix is never written
