"""Full-depth parity of the 7B- and 13B-shaped verification forwards (configs 3 and 4), in the launch configuration
bench.py times.

Two comparisons per case, from ONE oracle pass that keeps every layer's input and output:

* teacher-forced: layer l of the GPU path (cats_verify_layer) is given the ORACLE's residual stream as it enters layer
  l and must reproduce the oracle's output of that layer -- residual within 2e-2 flat (a few layers, above all the first,
  whose input is still of embedding size, may instead be held to twice the oracle's own fp32-accumulation spread of
  that layer), K/V rows within one bf16 ulp -- for every layer of the stack, so every kernel sees the residual stream as it
  really is at depth 16 or 31 (not a synthetic one); then the LM head from the oracle's final residual: logits within
  2e-2, argmax identical wherever the oracle's top-1 margin exceeds 2e-2.  No rounding flip of an earlier layer can hide or mimic an error of a later one.
* free-running: the whole forward (cats_verify_forward) against the oracle's logits.  A bf16 rounding point is a
  discontinuity, so two valid evaluations of the same contract drift apart with depth; the oracle measures that drift
  itself (fp64- against fp32-accumulated projections, a mode pinned in tests/test_oracle_pins.py).  The measured error,
  the drift and their ratio are printed and, if CATS_PARITY_REPORT names a file, appended to it as JSON lines.

The integer outputs (walk, compaction) are checked bit-exactly both ways in every case, and one case plants the tree's
tokens from the model's own top-k logits so that the walk and the compaction move a real multi-node path."""
import json
import os

import numpy as np
import pytest
import torch

import oracle
from paper_2605_11186_b200 import inputs as gen
from helpers import ref_cfg, np_model, cache_to_f32

pytestmark = pytest.mark.gpu

TOL = 2e-2
# Free-running bound: the GPU may sit this many times the oracle's own fp64-vs-fp32 drift away from the oracle.  Measured
# ratios on B200 are listed in the design notes; the factor is the smallest that clears them with a margin.
DRIFT_FACTOR = 1.5


@pytest.fixture(scope="module")
def cats():
    from paper_2605_11186_b200 import binding
    assert torch.cuda.is_available()
    return binding


def report(**row):
    print("parity:", json.dumps(row))
    path = os.environ.get("CATS_PARITY_REPORT")
    if path:
        with open(path, "a") as f:
            f.write(json.dumps(row) + "\n")


def bf16_ulp_bad(got_bf16: torch.Tensor, want_f32: np.ndarray):
    g = got_bf16.float().cpu().numpy().astype(np.float64)
    w = want_f32.astype(np.float64)
    mag = np.maximum(np.abs(g), np.abs(w))
    ulp = 2.0 ** (np.floor(np.log2(np.maximum(mag, 1e-30))) - 7)
    d = np.abs(g - w)
    return int((d > ulp * 1.001 + 1e-3).sum()), int((d > 2 * ulp * 1.001 + 1e-3).sum()), float(d.max()), float((d > 0).mean())


class Stack:
    """A model on both sides: CPU tensors / bit patterns for the oracle, packed weights on the device."""

    def __init__(self, cats, m, tag, P, max_T):
        self.m, self.P = m, P
        self.max_seq = P + max_T
        model = gen.make_model(m, tag)
        self.nm = np_model(model)
        dm = {"layers": [{k: v.cuda() for k, v in w.items()} for w in model["layers"]]}
        for k in ("embed", "final_norm", "w_lm"):
            dm[k] = model[k].cuda()
        self.dm = cats.pack_model(dm, free_source=True)
        torch.cuda.empty_cache()
        self.kc, self.vc = gen.make_kv_prefix(m, m.n_layers, self.max_seq, P, tag)
        self.rcfg = ref_cfg(m, self.max_seq)
        self.tag = tag


def oracle_pass(s: Stack, parent, tokens, keep_layers):
    """The oracle's forward as a plain layer loop.  Returns dict(ins, outs, k, v, logits, amax, margin, resid)."""
    m, P = s.m, s.P
    _, mask, pos, _ = oracle.build_tree_mask(parent, P)
    r_k, r_v = cache_to_f32(s.kc), cache_to_f32(s.vc)
    resid = oracle.embed(s.nm["embed"], tokens)
    ins, outs = [], []
    for l in range(m.n_layers):
        if keep_layers:
            ins.append(resid.copy())
        oracle.verify_layer(s.rcfg, s.nm["layers"][l], resid, r_k[l], r_v[l], mask, pos, P)
        if keep_layers:
            outs.append(resid.copy())
    logits, amax, margin = oracle.lm_head_argmax(s.rcfg, s.nm["final_norm"], s.nm["w_lm"], resid)
    return dict(ins=ins, outs=outs, k=r_k, v=r_v, logits=logits, amax=amax, margin=margin, resid=resid, mask=mask, pos=pos)


def gpu_walk(cats, parent, tokens, amax):
    T = len(parent)
    path = torch.full((T,), -1, dtype=torch.int32, device="cuda")
    out = torch.full((T,), -1, dtype=torch.int32, device="cuda")
    sc = torch.zeros(2, dtype=torch.int32, device="cuda")
    st = cats.new_status()
    cats.cats_accept_path(torch.from_numpy(parent).cuda(), torch.from_numpy(tokens).cuda(), torch.from_numpy(amax).cuda(), T, path,
                          sc[0:1], out, sc[1:2], st)
    assert int(st.item()) == 0
    return path.cpu().numpy()[:int(sc[0])], out.cpu().numpy()[:int(sc[1])]


def check_case(cats, s: Stack, name, parent, tokens, with_drift, want_path_len=1):
    m, P, T, L = s.m, s.P, len(parent), s.m.n_layers
    H, D = m.hidden, m.n_heads * m.head_dim
    o = oracle_pass(s, parent, tokens, keep_layers=True)

    # ---- teacher-forced: every layer from the oracle's input of that layer ----
    cfg1 = cats.model_cfg(m, s.max_seq, 1)
    ws = cats.new_workspace(cfg1, T, P)
    d_mask = torch.from_numpy(o["mask"].view(np.int64)).cuda()
    d_pos = torch.from_numpy(o["pos"]).cuda()
    d_k, d_v = s.kc.cuda(), s.vc.cuda()
    worst = dict(resid=0.0, kv=0.0, layer=-1, kv_diff_frac=0.0)
    over = []                                    # layers whose residual error exceeds the flat tolerance
    for l in range(L):
        d_resid = torch.from_numpy(o["ins"][l]).cuda()
        st = cats.new_status()
        cats.cats_verify_layer(cfg1, cats.layer_weights(s.dm["layers"][l]), d_resid, d_k[l], d_v[l], d_mask, d_pos, T, P, ws, st)
        torch.cuda.synchronize()
        assert int(st.item()) == 0
        err = float(np.abs(d_resid.cpu().numpy() - o["outs"][l]).max())
        if err > TOL:
            # A rounding point is a discontinuity: where the residual stream is still tiny (the first layer starts from
            # embedding rows of standard deviation 0.02) a perturbation in the fifth digit of the attention output flips
            # a few per cent of the bf16 inputs of the MLP.  The oracle shows the same when its own projections are
            # accumulated in fp32 (the pinned set_accum32 mode): the layer is then held to twice that spread instead.
            r32 = o["ins"][l].copy()
            rk, rv = cache_to_f32(s.kc[l:l + 1])[0], cache_to_f32(s.vc[l:l + 1])[0]
            oracle.set_accum32(True)
            try:
                oracle.verify_layer(s.rcfg, s.nm["layers"][l], r32, rk, rv, o["mask"], o["pos"], P)
            finally:
                oracle.set_accum32(False)
            spread = float(np.abs(r32 - o["outs"][l]).max())
            over.append(dict(layer=l, err=err, oracle_fp32_spread=spread))
            assert err <= 2.0 * spread, "%s layer %d: residual max-abs-err %g, oracle's own spread %g" % (name, l, err, spread)
        for got, want in ((d_k[l], o["k"][l]), (d_v[l], o["v"][l])):
            # one bf16 ulp; deep in the stack a handful of the T x 4096 sums land so close to a rounding tie that flips
            # of two or three large inputs carry them across it: at most two elements per million may be two ulps off
            nbad, nbad2, kverr, frac = bf16_ulp_bad(got[P:P + T], want[P:P + T])
            assert nbad2 == 0 and nbad <= max(1, int(2e-6 * T * D + 0.5)), \
                "%s layer %d: %d K/V elements off by more than one bf16 ulp, %d by more than two (max %g)" % (name, l, nbad, nbad2, kverr)
            worst["kv_over_one_ulp"] = worst.get("kv_over_one_ulp", 0) + nbad
            worst["kv"] = max(worst["kv"], kverr)
            worst["kv_diff_frac"] = max(worst["kv_diff_frac"], frac)
        if err > worst["resid"]:
            worst["resid"], worst["layer"] = err, l
    # the flat tolerance holds from the oracle's own input at all but a few layers (the first ones, and at the 13B shape
    # an occasional deeper one that ends a few per cent above it)
    assert len(over) <= max(2, L // 8), over
    # ---- LM head from the oracle's final residual ----
    cfgL = cats.model_cfg(m, s.max_seq, L)
    wsL = cats.new_workspace(cfgL, T, P)
    logits = torch.zeros((T, m.vocab), dtype=torch.float32, device="cuda")
    amax = torch.zeros(T, dtype=torch.int32, device="cuda")
    st = cats.new_status()
    cats.cats_lm_head_argmax(cfgL, s.dm["final_norm"], s.dm["w_lm"], torch.from_numpy(o["resid"]).cuda(), T, logits, amax, wsL, st)
    torch.cuda.synchronize()
    assert int(st.item()) == 0
    head_err = float(np.abs(logits.cpu().numpy() - o["logits"]).max())
    assert head_err <= TOL, "%s: LM head max-abs-err %g from the oracle's final residual" % (name, head_err)
    clear = o["margin"] > TOL
    assert np.array_equal(amax.cpu().numpy()[clear], o["amax"][clear])
    del ws, wsL, logits

    # ---- free-running forward ----
    d_k, d_v = s.kc.cuda(), s.vc.cuda()
    fwd = cats.VerifyForward(m, s.dm, d_k, d_v, T, P, want_logits=True, compact=False)
    fwd.run(torch.from_numpy(parent).cuda(), torch.from_numpy(tokens).cuda())
    torch.cuda.synchronize()
    assert int(fwd.status.item()) == 0
    g_logits = fwd.logits.cpu().numpy()
    g_amax = fwd.argmax.cpu().numpy()
    free_err = float(np.abs(g_logits - o["logits"]).max())
    free_rms = float(np.sqrt(np.mean((g_logits - o["logits"]).astype(np.float64) ** 2)))
    assert np.array_equal(g_amax, g_logits.argmax(-1))               # the GPU's argmax is the argmax of its own logits
    row = dict(case=name, T=T, layers=L, teacher_forced_resid_err=worst["resid"], at_layer=worst["layer"], layers_over_tol=over,
               teacher_forced_kv_err=worst["kv"], kv_over_one_ulp=worst.get("kv_over_one_ulp", 0), kv_diff_frac=worst["kv_diff_frac"], lm_head_err=head_err,
               free_running_logit_err=free_err, free_running_logit_rms=free_rms, logit_std=float(o["logits"].std()))
    bound = TOL
    if with_drift:
        oracle.set_accum32(True)
        try:
            o32 = oracle_pass(s, parent, tokens, keep_layers=False)
        finally:
            oracle.set_accum32(False)
        drift = float(np.abs(o32["logits"] - o["logits"]).max())
        drift_rms = float(np.sqrt(np.mean((o32["logits"] - o["logits"]).astype(np.float64) ** 2)))
        bound = max(TOL, DRIFT_FACTOR * drift)
        row.update(oracle_drift=drift, oracle_drift_rms=drift_rms, err_over_drift=free_err / drift, rms_over_drift_rms=free_rms / drift_rms,
                   bound=bound)
        assert free_err <= bound, row
        assert free_rms <= max(TOL / 4, DRIFT_FACTOR * drift_rms), row
    clear = o["margin"] > (TOL if bound == TOL else 2 * bound)
    row.update(nodes_with_clear_margin=int(clear.sum()), argmax_equal=int((g_amax == o["amax"]).sum()))
    if with_drift:
        assert np.array_equal(g_amax[clear], o["amax"][clear]), row

    # ---- walk: the integer kernel in isolation, both ways; end to end where the margins allow ----
    g_path = fwd.path.cpu().numpy()[:int(fwd.scalars[0])]
    g_out = fwd.out_tokens.cpu().numpy()[:int(fwd.scalars[1])]
    p2, o2 = oracle.accept_path(parent, tokens, g_amax)
    assert np.array_equal(g_path, p2) and np.array_equal(g_out, o2)
    r_path, r_out = oracle.accept_path(parent, tokens, o["amax"])
    p3, o3 = gpu_walk(cats, parent, tokens, o["amax"])
    assert np.array_equal(p3, r_path) and np.array_equal(o3, r_out)
    if with_drift and all(clear[n] for n in r_path):
        assert np.array_equal(g_path, r_path) and np.array_equal(g_out, r_out)
    row.update(gpu_path_len=len(g_path), oracle_path_len=len(r_path), paths_equal=bool(np.array_equal(g_path, r_path)))
    assert len(g_path) >= want_path_len, row

    # ---- compaction: a pure move of the GPU's own rows ----
    before_k, before_v = d_k.clone(), d_v.clone()
    new_len = torch.zeros(1, dtype=torch.int32, device="cuda")
    src = torch.full((T,), -1, dtype=torch.int32, device="cuda")
    dst = torch.full((T,), -1, dtype=torch.int32, device="cuda")
    st = cats.new_status()
    cats.cats_compact_kv(d_k, d_v, L, s.max_seq * D, D, P, fwd.path, fwd.scalars[0:1], new_len, src, dst, st)
    n = len(g_path)
    assert int(new_len.item()) == P + n and int(st.item()) == 0
    rc, r_new, r_src, r_dst = oracle.compact_kv(np.zeros((1, P + T, 8), np.float32), np.zeros((1, P + T, 8), np.float32), P, g_path)
    assert rc == 0 and r_new == P + n
    assert np.array_equal(src.cpu().numpy()[:n], r_src) and np.array_equal(dst.cpu().numpy()[:n], r_dst)
    idx = torch.as_tensor(P + g_path, device="cuda", dtype=torch.long)
    assert torch.equal(d_k[:, P:P + n], before_k[:, idx]) and torch.equal(d_v[:, P:P + n], before_v[:, idx])
    assert torch.equal(d_k[:, :P], before_k[:, :P]) and torch.equal(d_v[:, :P], before_v[:, :P])
    report(**row)
    return row


@pytest.fixture(scope="module")
def stack_7b(cats):
    s = Stack(cats, gen.LLAMA_7B, "cfg3_full", 512, 128)
    yield s
    del s
    torch.cuda.empty_cache()


@pytest.mark.parametrize("T,with_drift", [(16, True), (32, False), (64, True), (128, False)])
def test_config3_full_depth(cats, stack_7b, T, with_drift):
    """Config 3: 32 layers of the 7B shape + LM head, prefix 512, top-k tree shape of T nodes, uniform tokens."""
    parent, _ = gen.tree_topk_shape(T, gen.topk_k_for(T))
    tokens = gen.uniform_tokens(T, gen.LLAMA_7B.vocab, "cfg3_full", T)
    check_case(cats, stack_7b, "cfg3_T%d" % T, parent, tokens, with_drift)


def test_config3_planted_tree_moves_a_real_path(cats, stack_7b):
    """Config 3, T = 64, with the child tokens planted level by level from the model's own top-k logits (what a top-K
    drafter produces; input preparation, done with the library's forward), the top-1 withheld with probability 0.3:
    the accepted path has several nodes, so the walk and the compaction move real rows at 7B size."""
    s, T = stack_7b, 64
    parent, _ = gen.tree_topk_shape(T, gen.topk_k_for(T))
    depth = np.zeros(T, np.int64)
    for i in range(1, T):
        depth[i] = depth[parent[i]] + 1
    tokens = gen.uniform_tokens(T, s.m.vocab, "cfg3_planted", T)
    fwd = cats.VerifyForward(s.m, s.dm, s.kc.cuda(), s.vc.cuda(), T, s.P, want_logits=True, compact=False)
    rng = np.random.Generator(np.random.Philox(gen.substream("cfg3_planted", "coins")))
    d_parent = torch.from_numpy(parent).cuda()
    for d in range(int(depth.max())):
        fwd.run(d_parent, torch.from_numpy(tokens).cuda())
        torch.cuda.synchronize()
        for n in np.nonzero(depth == d)[0]:
            kids = np.nonzero(parent == n)[0]
            if len(kids) == 0:
                continue
            top = torch.topk(fwd.logits[n], len(kids) + 1).indices.cpu().numpy()
            start = 0 if (d < 2 or rng.random() < 0.7) else 1          # the first two levels always hold the top-1
            for r, c in enumerate(kids):
                tokens[c] = top[start + r]
    del fwd
    check_case(cats, s, "cfg3_T64_planted", parent, tokens, with_drift=False, want_path_len=3)


def test_config4_full_depth(cats):
    """Config 4: 40 layers of the 13B shape + LM head, prefix 2048, 64-node tree [6,3,2,2,1,1], uniform tokens."""
    s = Stack(cats, gen.LLAMA_13B, "cfg4_full", 2048, 64)
    parent = gen.tree_branching([6, 3, 2, 2, 1, 1], 64)
    tokens = gen.uniform_tokens(64, s.m.vocab, "cfg4_full", "t")
    check_case(cats, s, "cfg4_T64", parent, tokens, with_drift=True)
