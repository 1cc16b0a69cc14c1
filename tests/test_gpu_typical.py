"""GPU parity of typical (relaxed) acceptance: the softmax statistics the LM-head kernel leaves behind, the walk's verdicts
(bit-exact: both sides take them in fp32 in the same operation order) and the whole forward in typical mode."""
import math

import numpy as np
import pytest
import torch

import oracle
from paper_2605_11186_b200 import inputs as gen
from helpers import ref_cfg, np_model, cache_to_f32, oracle_prefill, planted_tree
from test_gpu_parity import TOL, dev, dev_model

pytestmark = pytest.mark.gpu

TEMP, EPS, DELTA = 0.7, 0.09, 0.3
INV_T = np.float32(1.0) / np.float32(TEMP)
LOG_EPS, LOG_DELTA = np.float32(math.log(EPS)), np.float32(math.log(DELTA))


@pytest.fixture(scope="module")
def cats():
    from paper_2605_11186_b200 import binding
    assert torch.cuda.is_available()
    return binding


def _gpu_walk_typical(cats, parent, tokens, amax, cand, lse, ent, inv_t=INV_T, log_eps=LOG_EPS, log_delta=LOG_DELTA):
    T = len(parent)
    path = torch.full((T,), -1, dtype=torch.int32, device="cuda")
    out = torch.full((T,), -1, dtype=torch.int32, device="cuda")
    n = torch.zeros(2, dtype=torch.int32, device="cuda")
    st = cats.new_status()
    cats.cats_accept_path_typical(dev(parent), dev(tokens), dev(amax), dev(cand), dev(lse), dev(ent), T, inv_t, log_eps,
                                  log_delta, path, n[0:1], out, n[1:2], st)
    torch.cuda.synchronize()
    assert int(st.item()) == 0
    pl, no = int(n[0]), int(n[1])
    return path.cpu().numpy()[:pl], out.cpu().numpy()[:no]


def test_walk_verdicts_are_bit_exact_on_random_and_near_threshold_inputs(cats):
    rng = np.random.default_rng(21)
    lengths = set()
    for trial in range(150):
        T = int(rng.integers(1, 129))
        parent = gen.tree_random(T, 300 + trial) if trial % 3 else gen.tree_chain(T)
        V = 50
        tokens = rng.integers(0, V, T).astype(np.int32)
        amax = rng.integers(0, V, T).astype(np.int32)
        lse = (rng.standard_normal(T) * 2 + 5).astype(np.float32)
        ent = np.abs(rng.standard_normal(T) * 1.5).astype(np.float32)
        # candidate logits placed so that fma(cand, 1/t, -lse) lands within a few ulps of the threshold for most nodes
        pa = np.maximum(parent, 0)
        thr = np.minimum(LOG_EPS, (LOG_DELTA - ent[pa]).astype(np.float32))
        cand = ((thr + lse[pa]) / INV_T).astype(np.float32)
        steps = rng.integers(-3, 4, T)
        for _ in range(3):
            cand = np.where(steps > 0, np.nextafter(cand, np.float32(np.inf)), np.where(steps < 0, np.nextafter(cand, np.float32(-np.inf)), cand))
            steps = steps - np.sign(steps)
        far = rng.random(T) < 0.3
        cand = np.where(far, cand + rng.standard_normal(T).astype(np.float32), cand).astype(np.float32)
        want = oracle.accept_path_typical(parent, tokens, amax, cand, lse, ent, INV_T, LOG_EPS, LOG_DELTA)
        got = _gpu_walk_typical(cats, parent, tokens, amax, cand, lse, ent)
        assert np.array_equal(got[0], want[0]) and np.array_equal(got[1], want[1]), trial
        lengths.add(len(want[0]))
    assert len(lengths) >= 5


def _head_case(cats, m, T, resid_std, tag, parent, tokens):
    resid = gen.normal_bf16((T, m.hidden), resid_std, "cpu", tag, "resid").float() + 1e-3 * gen.normal_bf16((T, m.hidden), 1.0, "cpu", tag, "lo").float()
    gain = (1.0 + gen.normal_bf16((m.hidden,), 0.2, "cpu", tag, "g").float()).to(torch.bfloat16)
    w_lm = gen.normal_bf16((m.vocab, m.hidden), 0.02, "cpu", tag, "w")
    rcfg = oracle.RefCfg(m.hidden, m.n_heads, m.head_dim, m.ffn, m.vocab, 0, 256, m.rms_eps, m.rope_base)
    logits, amax, margin = oracle.lm_head_argmax(rcfg, gen.bf16_bits(gain), gen.bf16_bits(w_lm), resid.numpy())
    cfg = cats.model_cfg(m, 256, 0)
    ws = cats.new_workspace(cfg, T, 0)
    d_logits = torch.zeros((T, m.vocab), dtype=torch.float32, device="cuda")
    d_amax = torch.zeros(T, dtype=torch.int32, device="cuda")
    stats = torch.full((3, T), 7.0, dtype=torch.float32, device="cuda")
    st = cats.new_status()
    cats.cats_lm_head_typical(cfg, gain.cuda(), cats.pack_weights([w_lm.cuda()], 0), resid.cuda(), dev(parent), dev(tokens), T,
                              INV_T, d_logits, d_amax, stats[0], stats[1], stats[2], ws, st)
    torch.cuda.synchronize()
    assert int(st.item()) == 0
    g = d_logits.cpu().numpy()
    assert np.abs(g - logits).max() <= TOL
    assert np.array_equal(d_amax.cpu().numpy(), g.argmax(-1))
    g_lse, g_ent, g_cand = (x.cpu().numpy() for x in stats)
    # on identical inputs (the GPU's own logits): the definitions in fp64
    lse, ent, cand, _ = oracle.typical_stats(g, float(1.0 / INV_T), parent, tokens)
    assert np.array_equal(g_cand, cand)                       # the very accumulator that was written as the logit
    assert np.abs(g_lse - lse).max() <= 1e-4 * max(1.0, np.abs(lse).max())
    assert np.abs(g_ent - ent).max() <= 2e-4 * max(1.0, np.abs(ent).max())
    # against the oracle's own logits: the logit tolerance, scaled by 1/t
    lse_o, ent_o, cand_o, _ = oracle.typical_stats(logits, float(1.0 / INV_T), parent, tokens)
    assert np.abs(g_lse - lse_o).max() <= TOL * float(INV_T) + 1e-3
    assert np.abs(g_cand - cand_o).max() <= TOL
    assert np.abs(g_ent - ent_o).max() <= 0.1
    return g, d_amax.cpu().numpy(), (g_lse, g_ent, g_cand)


def test_lm_head_statistics_tiny_ragged_vocabulary(cats):
    m = gen.TINY.replace(n_layers=0)
    for T, seed in [(1, 0), (37, 1), (128, 2)]:
        parent = gen.tree_random(T, seed)
        tokens = gen.uniform_tokens(T, m.vocab, "typ_head", T)
        _head_case(cats, m, T, 3.0, ("typ_tiny", T), parent, tokens)


def test_lm_head_statistics_7b_shape(cats):
    m = gen.LLAMA_7B.replace(n_layers=0)
    T = 64
    parent, _ = gen.tree_topk_shape(T, 10)
    tokens = gen.uniform_tokens(T, m.vocab, "typ_head7b", T)
    tokens[5] = m.vocab - 1                                    # last row of the last vocabulary tile
    tokens[6] = 0
    g, amax, (lse, ent, cand) = _head_case(cats, m, T, 3.0, "typ_7b", parent, tokens)
    # the walk on these statistics, GPU against the fixed-precision oracle walk
    want = oracle.accept_path_typical(parent, tokens, amax, cand, lse, ent, INV_T, LOG_EPS, LOG_DELTA)
    got = _gpu_walk_typical(cats, parent, tokens, amax, cand, lse, ent)
    assert np.array_equal(got[0], want[0]) and np.array_equal(got[1], want[1])


@pytest.fixture(scope="module")
def cfg1():
    m = gen.TINY
    model = gen.make_model(m, "cfg1")
    P, max_seq = 128, 320
    nm = np_model(model)
    rcfg = ref_cfg(m, max_seq)
    kc = np.zeros((m.n_layers, max_seq, m.n_heads * m.head_dim), np.float32)
    vc = np.zeros_like(kc)
    prompt = gen.uniform_tokens(P, m.vocab, "cfg1", "prompt")
    root = oracle_prefill(rcfg, nm, prompt, kc, vc)
    return dict(m=m, model=model, nm=nm, rcfg=rcfg, kc=kc, vc=vc, P=P, max_seq=max_seq, root=root)


@pytest.mark.parametrize("T,k,seed,temp", [(16, 4, 0, 0.7), (32, 4, 2, 0.7), (40, 10, 3, 0.7), (128, 10, 4, 0.7), (32, 4, 5, 0.05)])
def test_whole_forward_in_typical_mode(cats, cfg1, T, k, seed, temp):
    """Tiny model, planted top-k trees.  The tiny model's distributions are nearly flat (logit std 0.3) at t = 0.7, so
    most children pass; t = 0.05 sharpens them so that the criterion also rejects."""
    c = cfg1
    m = c["m"]
    nm = c["nm"]
    inv_t = np.float32(1.0) / np.float32(temp)
    parent, tokens = planted_tree(c["rcfg"], nm, T, k, c["root"], c["P"], c["kc"], c["vc"], (seed,))
    r_k, r_v = c["kc"].copy(), c["vc"].copy()
    logits, amax, margin, _ = oracle.verify_forward(c["rcfg"], nm["layers"], nm["embed"], nm["final_norm"], nm["w_lm"], parent,
                                                    tokens, c["P"], r_k, r_v)
    dm = cats.pack_model(dev_model(c["model"]))
    d_k = torch.from_numpy(c["kc"]).to(torch.bfloat16).cuda()
    d_v = torch.from_numpy(c["vc"]).to(torch.bfloat16).cuda()
    before_k = d_k.clone()
    fwd = cats.VerifyForward(m, dm, d_k, d_v, T, c["P"], want_logits=True, compact=True, typical=(inv_t, LOG_EPS, LOG_DELTA))
    fwd.run(dev(parent), dev(tokens))
    torch.cuda.synchronize()
    assert int(fwd.status.item()) == 0
    g_logits = fwd.logits.cpu().numpy()
    assert np.abs(g_logits - logits).max() <= TOL
    g_amax = fwd.argmax.cpu().numpy()
    g_lse, g_ent, g_cand = (x.cpu().numpy() for x in fwd.typical)
    g_path = fwd.path.cpu().numpy()[:int(fwd.scalars[0])]
    g_out = fwd.out_tokens.cpu().numpy()[:int(fwd.scalars[1])]
    # (1) the walk, bit-exact, on the statistics the GPU produced
    want = oracle.accept_path_typical(parent, tokens, g_amax, g_cand, g_lse, g_ent, inv_t, LOG_EPS, LOG_DELTA)
    assert np.array_equal(g_path, want[0]) and np.array_equal(g_out, want[1])
    # (2) the statistics against the definition on the GPU's own logits
    lse, ent, cand, prob = oracle.typical_stats(g_logits, float(temp), parent, tokens)
    assert np.array_equal(g_cand, cand)
    assert np.abs(g_lse - lse).max() <= 1e-4 * max(1.0, np.abs(lse).max()) and np.abs(g_ent - ent).max() <= 2e-4 * max(1.0, np.abs(ent).max())
    # (3) the path the definition gives on the ORACLE's logits, wherever no verdict on it is close to its threshold
    _, ent_o, _, prob_o = oracle.typical_stats(logits, float(temp), parent, tokens)
    thr_o = np.minimum(EPS, DELTA * np.exp(-ent_o.astype(np.float64)))[np.maximum(parent, 0)]
    gap = np.abs(np.log(np.maximum(prob_o, 1e-300)) - np.log(thr_o))
    r_path, r_out = oracle.accept_path_typical_def(parent, tokens, amax, logits, float(temp), EPS, DELTA)
    touched = [j for j in range(1, T) if parent[j] in set(r_path.tolist())]
    if all(gap[j] > 5 * TOL * float(inv_t) for j in touched) and margin[r_path[-1]] > TOL:
        assert np.array_equal(g_path, r_path) and np.array_equal(g_out, r_out)
    # (4) roll-back along the accepted path
    n = len(g_path)
    assert int(fwd.scalars[2]) == c["P"] + n
    idx = torch.as_tensor(c["P"] + g_path, device="cuda", dtype=torch.long)
    assert torch.equal(d_k[:, :c["P"]], before_k[:, :c["P"]])
    assert d_k[:, c["P"]:c["P"] + n].abs().sum() > 0
    assert n >= 1 and g_path[0] == 0
