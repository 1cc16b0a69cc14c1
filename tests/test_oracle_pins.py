"""Pins of the CPU oracle against things other than itself: brute force, closed forms, torch float64
library routines, a HuggingFace LLaMA forward with an explicit 4-D mask, and Algorithm 1's own walk."""
import itertools
import math

import numpy as np
import pytest
import torch
import torch.nn.functional as F

import oracle
from paper_2605_11186_b200 import inputs as gen
from helpers import ref_cfg, np_model, oracle_prefill, oracle_greedy_decode, planted_tree


@pytest.fixture(autouse=True)
def _contract_on():
    oracle.set_contract(True)
    yield
    oracle.set_contract(True)


# ---------------------------------------------------------------------------------------------------
# bf16 rounding helper against torch's conversion
# ---------------------------------------------------------------------------------------------------

def test_bf16_round_matches_torch():
    rng = np.random.default_rng(1)
    x = np.concatenate([rng.standard_normal(20000).astype(np.float32) * s for s in (1e-3, 1.0, 300.0)])
    # ties: values exactly halfway between two bf16 numbers
    base = np.array([1.0, 1.0078125, 2.5, -3.0, 0.02], np.float32)
    halfway = (oracle.from_bf16(oracle.to_bf16(base)).view(np.uint32) | 0x8000).view(np.float32)
    x = np.concatenate([x, halfway, np.array([0.0, -0.0, np.inf, -np.inf], np.float32)])
    want = torch.from_numpy(x).to(torch.bfloat16).view(torch.int16).numpy().view(np.uint16)
    got = oracle.to_bf16(x)
    assert np.array_equal(got, want)
    assert np.array_equal(oracle.from_bf16(got), torch.from_numpy(x).to(torch.bfloat16).float().numpy())
    # the C helper used inside the forward agrees with the vectorised one
    for v in x[:200]:
        assert oracle.ref._lib.cats_ref_f32_to_bf16(float(v)) == int(oracle.to_bf16(np.array([v]))[0])


# ---------------------------------------------------------------------------------------------------
# P1: ancestor mask against brute force, exhaustively for all trees of up to 8 nodes
# ---------------------------------------------------------------------------------------------------

def _closure_mask(parent):
    """Reflexive-transitive closure of the child->parent relation by boolean matrix powers."""
    n = len(parent)
    A = np.eye(n, dtype=np.int64)
    for i in range(1, n):
        A[i, parent[i]] = 1
    R = A
    for _ in range(max(1, int(np.ceil(np.log2(max(n, 2)))))):   # repeated squaring, clipped to 0/1
        R = ((R @ R) > 0).astype(np.int64)
    return R > 0


def test_mask_exhaustive_up_to_8_nodes():
    count = 0
    for n in range(1, 9):
        for combo in itertools.product(*[range(i) for i in range(1, n)]):
            parent = np.array((-1,) + combo, np.int32)
            rc, mask, pos, depth = oracle.build_tree_mask(parent, 5)
            assert rc == 0
            want = _closure_mask(parent)
            got = np.array([[(int(mask[i, j >> 6]) >> (j & 63)) & 1 for j in range(n)] for i in range(n)], bool)
            assert np.array_equal(got, want), parent
            assert mask[:, 1].max() == 0 and all(int(mask[i, 0]) >> n == 0 for i in range(n))
            # depth = number of proper ancestors; pos = prefix + depth
            assert np.array_equal(depth, want.sum(1) - 1)
            assert np.array_equal(pos, 5 + depth)
            count += 1
    assert count == sum(math.factorial(n - 1) for n in range(1, 9))


def test_mask_large_trees_cross_word_boundary():
    for parent in (gen.tree_chain(128), gen.tree_heap(64), gen.tree_random(128, 3), gen.tree_branching([8, 4, 2, 1, 1], 64)):
        rc, mask, pos, depth = oracle.build_tree_mask(parent, 1000)
        assert rc == 0
        want = _closure_mask(parent)
        n = len(parent)
        got = np.array([[(int(mask[i, j >> 6]) >> (j & 63)) & 1 for j in range(n)] for i in range(n)], bool)
        assert np.array_equal(got, want)
        assert np.array_equal(pos, 1000 + want.sum(1) - 1)


def test_mask_rejects_malformed_trees():
    assert oracle.build_tree_mask(np.array([0, 0], np.int32), 0)[0] == -2
    assert oracle.build_tree_mask(np.array([-1, 1], np.int32), 0)[0] == -2
    assert oracle.build_tree_mask(np.array([-1, 0, 3, 1], np.int32), 0)[0] == -2
    assert oracle.build_tree_mask(np.array([-1, -1], np.int32), 0)[0] == -2


def test_tree_generators_shapes():
    # level sizes fixed by the branching lists
    for b, T, levels in (([4, 2, 1, 1], 16, [1, 4, 8, 3]), ([8, 4, 2, 1, 1], 64, [1, 8, 32, 23]),
                         ([6, 3, 2, 2, 1, 1], 64, [1, 6, 18, 36, 3])):
        parent = gen.tree_branching(b, T)
        _, _, _, depth = oracle.build_tree_mask(parent, 0)
        assert [int((depth == d).sum()) for d in range(len(levels))] == levels
    assert np.array_equal(gen.tree_chain(4), [-1, 0, 1, 2])
    assert np.array_equal(gen.tree_heap(6), [-1, 0, 0, 0, 0, 1])
    p = gen.tree_random(128, 0)
    kids = np.bincount(p[1:], minlength=128)
    assert kids.max() <= 4 and p[0] == -1 and all(p[i] < i for i in range(1, 128))


# ---------------------------------------------------------------------------------------------------
# P6: single ops against torch float64 library routines (pure mode: no bf16 rounding)
# ---------------------------------------------------------------------------------------------------

def test_rmsnorm_matches_torch():
    oracle.set_contract(False)
    rng = np.random.default_rng(2)
    x = rng.standard_normal((5, 96)).astype(np.float32) * 3
    g = oracle.to_bf16(rng.standard_normal(96).astype(np.float32))
    got = oracle.rmsnorm(x, g, 1e-5)
    want = F.rms_norm(torch.from_numpy(x).double(), (96,), torch.from_numpy(oracle.from_bf16(g)).double(), 1e-5)
    assert np.abs(got - want.numpy()).max() < 1e-12


def test_linear_matches_torch_matmul():
    rng = np.random.default_rng(3)
    W = oracle.to_bf16(rng.standard_normal((37, 129)).astype(np.float32))
    x = rng.standard_normal((7, 129))
    got = oracle.linear(W, x)
    want = torch.from_numpy(x) @ torch.from_numpy(oracle.from_bf16(W)).double().T
    assert np.abs(got - want.numpy()).max() < 1e-12
    # a transposed weight would fail: shapes differ, and a square case too
    Wsq = oracle.to_bf16(rng.standard_normal((16, 16)).astype(np.float32))
    xs = rng.standard_normal((3, 16))
    wf = torch.from_numpy(oracle.from_bf16(Wsq)).double()
    assert np.abs(oracle.linear(Wsq, xs) - (torch.from_numpy(xs) @ wf.T).numpy()).max() < 1e-12
    assert np.abs(oracle.linear(Wsq, xs) - (torch.from_numpy(xs) @ wf).numpy()).max() > 1e-3


def test_linear_fp32_accumulation_mode_is_a_sequential_float32_sum():
    """The oracle's fp32-accumulation mode (set_accum32) sets the noise floor that the deep-stack GPU tests report
    beside their errors, so it is pinned like any other function: every output must equal, bit for bit, a float32
    running sum over ascending k of separately rounded float32 products (written here with numpy scalars); and it must
    sit at the distance from the fp64 sum that float32 rounding of ~K terms predicts, not at zero and not far away."""
    rng = np.random.default_rng(33)
    n_out, K, T = 11, 300, 5
    W = oracle.to_bf16(rng.standard_normal((n_out, K)).astype(np.float32))
    x = rng.standard_normal((T, K))
    want64 = oracle.linear(W, x)
    oracle.set_accum32(True)
    try:
        got = oracle.linear(W, x)
    finally:
        oracle.set_accum32(False)
    Wf = oracle.from_bf16(W)
    xf = x.astype(np.float32)
    want = np.zeros((T, n_out), np.float32)
    for t in range(T):
        for o in range(n_out):
            acc = np.float32(0.0)
            for k in range(K):
                acc = np.float32(acc + np.float32(Wf[o, k] * xf[t, k]))
            want[t, o] = acc
    assert np.array_equal(got.astype(np.float32), want) and np.array_equal(got, want.astype(np.float64))
    # a descending-k or pairwise sum would differ in the last bits of most outputs
    rev = np.zeros((T, n_out), np.float32)
    for t in range(T):
        for o in range(n_out):
            acc = np.float32(0.0)
            for k in range(K - 1, -1, -1):
                acc = np.float32(acc + np.float32(Wf[o, k] * xf[t, k]))
            rev[t, o] = acc
    assert not np.array_equal(rev, want)
    # distance from the fp64 sum: inputs rounded to float32 plus ~K float32 additions of terms of size ~1
    d = np.abs(got - want64).max()
    assert 1e-7 < d < 2e-4, d
    assert np.array_equal(oracle.linear(W, x), want64)      # the switch is off again


def test_rope_closed_forms():
    rng = np.random.default_rng(4)
    hd = 64
    x = rng.standard_normal(hd)
    y = rng.standard_normal(hd)
    # position 0 is the identity
    assert np.array_equal(oracle.rope_head(x, 0, 10000.0), x)
    # a rotation: pair norms are preserved
    r = oracle.rope_head(x, 37, 10000.0)
    assert np.allclose(r[:32] ** 2 + r[32:] ** 2, x[:32] ** 2 + x[32:] ** 2, rtol=1e-12)
    # pair i turns by the angle pos * base^(-2i/hd), counter-clockwise
    for i in (0, 1, 17, 31):
        ang = 37 * 10000.0 ** (-2.0 * i / hd)
        z = complex(x[i], x[i + 32]) * complex(math.cos(ang), math.sin(ang))
        assert abs(r[i] - z.real) < 1e-12 and abs(r[i + 32] - z.imag) < 1e-12
    # relative property: <R_m q, R_n k> depends on m - n only
    a = np.dot(oracle.rope_head(x, 50, 10000.0), oracle.rope_head(y, 43, 10000.0))
    b = np.dot(oracle.rope_head(x, 1007, 10000.0), oracle.rope_head(y, 1000, 10000.0))
    assert abs(a - b) < 1e-9


def _bool_mask(mask, T, P):
    m = np.ones((T, P + T), bool)
    for i in range(T):
        for j in range(T):
            m[i, P + j] = (int(mask[i, j >> 6]) >> (j & 63)) & 1
    return m


@pytest.mark.parametrize("parent,P", [(gen.tree_branching([4, 2, 1, 1], 16), 19), (gen.tree_random(70, 1), 33),
                                      (gen.tree_chain(9), 0)])
def test_tree_attention_matches_torch_sdpa(parent, P):
    oracle.set_contract(False)
    T = len(parent)
    nh, hd = 3, 16
    rng = np.random.default_rng(5)
    q = rng.standard_normal((T, nh, hd))
    kc = rng.standard_normal((P + T, nh * hd)).astype(np.float32)
    vc = rng.standard_normal((P + T, nh * hd)).astype(np.float32)
    _, mask, _, _ = oracle.build_tree_mask(parent, P)
    got, probs = oracle.tree_attention(q, kc, vc, mask, P, nh, hd, 0.37, want_probs=True)
    bm = torch.from_numpy(_bool_mask(mask, T, P))
    tq = torch.from_numpy(q).permute(1, 0, 2)[None]
    tk = torch.from_numpy(kc).double().view(P + T, nh, hd).permute(1, 0, 2)[None]
    tv = torch.from_numpy(vc).double().view(P + T, nh, hd).permute(1, 0, 2)[None]
    want = F.scaled_dot_product_attention(tq, tk, tv, attn_mask=bm[None, None], scale=0.37)[0].permute(1, 0, 2)
    assert np.abs(got - want.numpy()).max() < 1e-12
    # P7: probabilities sum to one, masked columns are exactly zero
    assert np.abs(probs.sum(-1) - 1).max() < 1e-12
    assert np.all(probs[:, ~bm.numpy()] == 0.0)
    assert np.all(probs[:, bm.numpy()] > 0.0)


def test_attention_ignores_non_ancestors():
    """P7: appending a node that is nobody's ancestor changes no other node's output."""
    oracle.set_contract(False)
    rng = np.random.default_rng(6)
    parent = gen.tree_branching([3, 2, 1], 10)
    T, P, nh, hd = 10, 7, 2, 8
    q = rng.standard_normal((T + 1, nh, hd))
    kc = rng.standard_normal((P + T + 1, nh * hd)).astype(np.float32)
    vc = rng.standard_normal((P + T + 1, nh * hd)).astype(np.float32)
    _, m1, _, _ = oracle.build_tree_mask(parent, P)
    _, m2, _, _ = oracle.build_tree_mask(np.append(parent, 4).astype(np.int32), P)
    a = oracle.tree_attention(q[:T], kc, vc, m1, P, nh, hd, 0.5)
    b = oracle.tree_attention(q, kc, vc, m2, P, nh, hd, 0.5)
    assert np.array_equal(a, b[:T])


# ---------------------------------------------------------------------------------------------------
# whole forward against HuggingFace LLaMA in float64 (pure mode), tree given as an explicit 4-D mask
# ---------------------------------------------------------------------------------------------------

def _hf_model(model):
    from transformers import LlamaConfig, LlamaForCausalLM
    m = model["shape"]
    cfg = LlamaConfig(hidden_size=m.hidden, intermediate_size=m.ffn, num_hidden_layers=m.n_layers,
                      num_attention_heads=m.n_heads, num_key_value_heads=m.n_heads, head_dim=m.head_dim,
                      vocab_size=m.vocab, rms_norm_eps=m.rms_eps, rope_theta=m.rope_base,
                      max_position_embeddings=1024, attention_bias=False, mlp_bias=False,
                      tie_word_embeddings=False, attn_implementation="eager")
    hf = LlamaForCausalLM(cfg).double().eval()
    sd = {"model.embed_tokens.weight": model["embed"], "model.norm.weight": model["final_norm"],
          "lm_head.weight": model["w_lm"]}
    names = {"wq": "self_attn.q_proj", "wk": "self_attn.k_proj", "wv": "self_attn.v_proj", "wo": "self_attn.o_proj",
             "w_gate": "mlp.gate_proj", "w_up": "mlp.up_proj", "w_down": "mlp.down_proj",
             "attn_norm": "input_layernorm", "mlp_norm": "post_attention_layernorm"}
    for l, w in enumerate(model["layers"]):
        for k, n in names.items():
            sd["model.layers.%d.%s.weight" % (l, n)] = w[k]
    missing = hf.load_state_dict({k: v.double() for k, v in sd.items()}, strict=False)
    assert not [k for k in missing.missing_keys if "rotary" not in k]
    return hf


@pytest.fixture(scope="module")
def tiny():
    model = gen.make_model(gen.TINY, "tiny")
    # distinct norm gains so that a dropped or misplaced gain shows (the workloads use gains of 1)
    for l, w in enumerate(model["layers"]):
        for n in gen.LAYER_NORMS:
            w[n] = (1.0 + gen.normal_bf16((gen.TINY.hidden,), 0.2, "cpu", "gain", l, n).float()).to(torch.bfloat16)
    model["final_norm"] = (1.0 + gen.normal_bf16((gen.TINY.hidden,), 0.2, "cpu", "gain", "f").float()).to(torch.bfloat16)
    return model


@pytest.mark.parametrize("tree", ["branching", "random", "chain"])
def test_forward_matches_huggingface_llama(tiny, tree):
    oracle.set_contract(False)
    m = gen.TINY
    nm = np_model(tiny)
    P = 24
    parent = {"branching": gen.tree_branching([4, 2, 1, 1], 16), "random": gen.tree_random(40, 9),
              "chain": gen.tree_chain(12)}[tree]
    T = len(parent)
    prompt = gen.uniform_tokens(P, m.vocab, "hf_prompt")
    tokens = gen.uniform_tokens(T, m.vocab, "hf_tree", tree)
    cfg = ref_cfg(m, 128)
    kc = np.zeros((m.n_layers, 128, m.n_heads * m.head_dim), np.float32)
    vc = np.zeros_like(kc)
    oracle_prefill(cfg, nm, prompt, kc, vc)
    logits, amax, margin, _ = oracle.verify_forward(cfg, nm["layers"], nm["embed"], nm["final_norm"], nm["w_lm"],
                                                    parent, tokens, P, kc, vc)
    hf = _hf_model(tiny)
    _, mask, pos, _ = oracle.build_tree_mask(parent, P)
    S = P + T
    allow = np.zeros((S, S), bool)
    allow[:P, :P] = np.tril(np.ones((P, P), bool))
    allow[P:, :] = _bool_mask(mask, T, P)
    add = torch.zeros(1, 1, S, S, dtype=torch.float64).masked_fill_(~torch.from_numpy(allow), float("-inf"))
    ids = torch.from_numpy(np.concatenate([prompt, tokens]).astype(np.int64))[None]
    position_ids = torch.from_numpy(np.concatenate([np.arange(P), pos]).astype(np.int64))[None]
    with torch.no_grad():
        want = hf(input_ids=ids, attention_mask=add, position_ids=position_ids).logits[0, P:].numpy()
    err = np.abs(logits - want).max()
    assert err < 2e-5, err      # the library keeps its RoPE tables in fp32; everything else is fp64
    assert np.array_equal(amax, want.argmax(-1))
    if tree == "chain":
        # P2: a chain tree is ordinary causal decoding -- the library's own causal path, no mask given
        with torch.no_grad():
            causal = hf(input_ids=ids).logits[0, P:].numpy()
        assert np.abs(logits - causal).max() < 2e-5
        assert np.array_equal(pos, np.arange(P, P + T))


def test_contract_mode_stays_close_to_pure_mode(tiny):
    """Not a pin (the paper states no 16-bit tolerance): reports how far the bf16 rounding points move the logits."""
    m = gen.TINY
    nm = np_model(tiny)
    cfg = ref_cfg(m, 64)
    parent = gen.tree_branching([4, 2, 1, 1], 16)
    tokens = gen.uniform_tokens(16, m.vocab, "cp")
    out = []
    for contract in (True, False):
        oracle.set_contract(contract)
        kc = np.zeros((m.n_layers, 64, 256), np.float32)
        vc = np.zeros_like(kc)
        oracle_prefill(cfg, nm, gen.uniform_tokens(20, m.vocab, "cp_prompt"), kc, vc)
        out.append(oracle.verify_forward(cfg, nm["layers"], nm["embed"], nm["final_norm"], nm["w_lm"], parent,
                                         tokens, 20, kc, vc)[0])
    d = np.abs(out[0] - out[1]).max()
    assert 0 < d < 2e-2


# ---------------------------------------------------------------------------------------------------
# P9 argmax / margin
# ---------------------------------------------------------------------------------------------------

def test_argmax_ties_and_margin():
    m = gen.ModelShape(hidden=8, n_heads=1, head_dim=8, ffn=8, vocab=6, n_layers=0)
    cfg = ref_cfg(m, 8)
    g = oracle.to_bf16(np.ones(8, np.float32))
    W = np.zeros((6, 8), np.float32)
    W[1, 0] = 1.0
    W[3, 0] = 1.0      # rows 1 and 3 give identical logits: the lower index must win
    W[4, 0] = 0.5
    W[5, 0] = -2.0
    resid = np.zeros((2, 8), np.float32)
    resid[0, 0] = 2.0
    resid[1, 0] = -1.0  # negative input: row 5 wins alone
    logits, amax, margin = oracle.lm_head_argmax(cfg, g, oracle.to_bf16(W), resid)
    assert list(amax) == [1, 5]
    assert margin[0] == 0.0 and margin[1] > 0
    assert np.array_equal(amax, [int(np.flatnonzero(r == r.max())[0]) for r in logits])
    srt = np.sort(logits, axis=1)
    assert np.allclose(margin, srt[:, -1] - srt[:, -2])


# ---------------------------------------------------------------------------------------------------
# P4: the generic walk equals Algorithm 1's loop on CATS-shaped trees
# ---------------------------------------------------------------------------------------------------

def _alg1_walk(d, corr, p_main, p_corr, p_bonus_of_node):
    """Algorithm 1's acceptance loop with greedy Acc.  d: main draft tokens; corr: {i: token};
    p_main[i]: target argmax judging position i; the correction at i is judged by the same distribution
    (it is a sibling of d_i); returns (y_out, accepted node list)."""
    a = 0
    y = []
    nodes = [0]
    gamma = len(d)
    corr_nodes = {i: gamma + 1 + r for r, i in enumerate(sorted(corr))}
    for i in range(gamma):
        if d[i] == p_main[i]:
            a += 1
            y.append(d[i])
            nodes.append(i + 1)
        elif i in corr and corr[i] == p_corr[i]:
            a += 1
            y.append(corr[i])
            nodes.append(corr_nodes[i])
            break
        else:
            break
    y.append(p_bonus_of_node[nodes[-1]])
    return y, nodes


def test_walk_equals_algorithm1_on_cats_trees():
    rng = np.random.default_rng(7)
    V = 5                                     # small vocabulary so matches are frequent
    seen = set()
    for _ in range(3000):
        gamma = int(rng.integers(1, 11))
        d = rng.integers(0, V, gamma)
        positions = [i for i in range(gamma) if rng.random() < 0.4]
        corr = {}
        for i in positions:
            c = int(rng.integers(0, V - 1))
            corr[i] = c if c < d[i] else c + 1    # a correction differs from the draft token it corrects
        parent = gen.tree_cats(gamma, positions)
        T = len(parent)
        tokens = np.zeros(T, np.int32)
        tokens[1:gamma + 1] = d
        for r, i in enumerate(sorted(positions)):
            tokens[gamma + 1 + r] = corr[i]
        amax = rng.integers(0, V, T).astype(np.int32)
        for i in range(gamma):                # make long accepted prefixes and accepted corrections common
            u = rng.random()
            if u < 0.7:
                amax[i] = d[i]
            elif u < 0.85 and i in corr:
                amax[i] = corr[i]
        # position i is judged by the argmax at node i (the parent of d_i and of its correction)
        y, nodes = _alg1_walk(list(d), corr, amax[:gamma], amax[:gamma], amax)
        path, out = oracle.accept_path(parent, tokens, amax)
        assert list(path) == nodes and list(out) == y
        seen.add((len(out), nodes[-1] > gamma))
    assert (1, False) in seen and any(n >= 6 for n, _ in seen) and any(c for _, c in seen)


def test_walk_hand_cases():
    parent = gen.tree_cats(3, [1])           # root, d0 d1 d2, correction at position 1 (node 4, child of node 1)
    tokens = np.array([9, 10, 11, 12, 21], np.int32)
    # nothing accepted: only the bonus token comes out
    path, out = oracle.accept_path(parent, tokens, np.array([7, 7, 7, 7, 7], np.int32))
    assert list(path) == [0] and list(out) == [7]
    # whole chain accepted: gamma + 1 tokens
    path, out = oracle.accept_path(parent, tokens, np.array([10, 11, 12, 5, 6], np.int32))
    assert list(path) == [0, 1, 2, 3] and list(out) == [10, 11, 12, 5]
    # correction accepted at position 1: i + 2 tokens, bonus from the correction node
    path, out = oracle.accept_path(parent, tokens, np.array([10, 21, 12, 5, 6], np.int32))
    assert list(path) == [0, 1, 4] and list(out) == [10, 21, 6]
    # duplicate sibling tokens: the lowest node index is taken
    parent2 = np.array([-1, 0, 0, 1, 2], np.int32)
    tok2 = np.array([1, 5, 5, 8, 8], np.int32)
    path, out = oracle.accept_path(parent2, tok2, np.array([5, 8, 8, 3, 4], np.int32))
    assert list(path) == [0, 1, 3] and list(out) == [5, 8, 3]
    # P12: a one-node tree is ordinary decoding
    path, out = oracle.accept_path(np.array([-1], np.int32), np.array([3], np.int32), np.array([4], np.int32))
    assert list(path) == [0] and list(out) == [4]


# ---------------------------------------------------------------------------------------------------
# P5: compaction
# ---------------------------------------------------------------------------------------------------

def test_compaction_moves_rows_and_indices():
    rng = np.random.default_rng(8)
    L, S, R, P = 3, 40, 6, 11
    kc = rng.integers(0, 60000, (L, S, R)).astype(np.uint16)
    vc = rng.integers(0, 60000, (L, S, R)).astype(np.uint16)
    k0, v0 = kc.copy(), vc.copy()
    path = np.array([0, 2, 5, 17], np.int32)
    rc, new_len, src, dst = oracle.compact_kv(kc, vc, P, path)
    assert rc == 0 and new_len == P + 4
    assert list(src) == [11, 13, 16, 28] and list(dst) == [11, 12, 13, 14]
    assert np.array_equal(kc[:, :P], k0[:, :P]) and np.array_equal(vc[:, :P], v0[:, :P])
    assert np.array_equal(kc[:, P:new_len], k0[:, P + path]) and np.array_equal(vc[:, P:new_len], v0[:, P + path])
    # identity path: nothing changes
    kc, vc = k0.copy(), v0.copy()
    rc, new_len, src, dst = oracle.compact_kv(kc, vc, P, np.array([0, 1, 2], np.int32))
    assert rc == 0 and new_len == P + 3 and np.array_equal(kc, k0) and np.array_equal(vc, v0)
    # a path that is not strictly increasing from the root is refused
    assert oracle.compact_kv(kc, vc, P, np.array([0, 3, 2], np.int32))[0] == -2
    assert oracle.compact_kv(kc, vc, P, np.array([1, 2], np.int32))[0] == 0  # path[k] >= k holds; root check is the walk's


# ---------------------------------------------------------------------------------------------------
# P3 / P5 / P10 / P11 / P12 end to end on the tiny model
# ---------------------------------------------------------------------------------------------------

@pytest.fixture(scope="module")
def tiny_ctx():
    """Config 1: tiny random decoder, prefix of 128 uniform tokens prefilled by the oracle."""
    oracle.set_contract(True)
    m = gen.TINY
    model = gen.make_model(m, "cfg1")
    nm = np_model(model)
    P = 128
    max_seq = 320
    cfg = ref_cfg(m, max_seq)
    kc = np.zeros((m.n_layers, max_seq, m.n_heads * m.head_dim), np.float32)
    vc = np.zeros_like(kc)
    prompt = gen.uniform_tokens(P, m.vocab, "cfg1", "prompt")
    root = oracle_prefill(cfg, nm, prompt, kc, vc)
    return dict(m=m, nm=nm, cfg=cfg, kc=kc, vc=vc, P=P, root=root, prompt=prompt)


def _fwd(ctx, parent, tokens, kc=None, vc=None):
    kc = ctx["kc"].copy() if kc is None else kc
    vc = ctx["vc"].copy() if vc is None else vc
    nm = ctx["nm"]
    out = oracle.verify_forward(ctx["cfg"], nm["layers"], nm["embed"], nm["final_norm"], nm["w_lm"], parent, tokens,
                                ctx["P"], kc, vc)
    return out, kc, vc


@pytest.mark.parametrize("T,k,seed", [(16, 4, 0), (16, 4, 1), (32, 4, 2), (40, 10, 3), (24, 4, 4), (16, 4, 5)])
def test_tree_walk_equals_sequential_greedy(tiny_ctx, T, k, seed):
    """P3: the tokens the tree verification emits are the tokens plain greedy decoding emits, and the walk
    stops exactly where the tree no longer holds the next greedy token.  P5: the compacted cache equals the
    cache of that sequential decoding."""
    ctx = tiny_ctx
    nm, cfg, P = ctx["nm"], ctx["cfg"], ctx["P"]
    parent, tokens = planted_tree(cfg, nm, T, k, ctx["root"], P, ctx["kc"], ctx["vc"], (seed,))
    (logits, amax, margin, _), kc, vc = _fwd(ctx, parent, tokens)
    path, out = oracle.accept_path(parent, tokens, amax)
    greedy, gk, gv = oracle_greedy_decode(cfg, nm, ctx["root"], P, ctx["kc"], ctx["vc"], len(out))
    assert list(out) == greedy[:len(out)]
    last = path[-1]
    kids = np.nonzero(parent == last)[0]
    assert greedy[len(out) - 1] not in tokens[kids]
    # compaction: rows [P, new_len) equal the sequentially decoded cache rows, bit for bit
    L, S, D = kc.shape
    rc, new_len, src, dst = oracle.compact_kv(kc, vc, P, path)
    assert rc == 0 and new_len == P + len(path)
    assert np.array_equal(kc[:, :new_len], gk[:, :new_len]) and np.array_equal(vc[:, :new_len], gv[:, :new_len])


def test_planted_trees_cover_several_accept_lengths(tiny_ctx):
    ctx = tiny_ctx
    lens = set()
    for seed in range(8):
        parent, tokens = planted_tree(ctx["cfg"], ctx["nm"], 16, 4, ctx["root"], ctx["P"], ctx["kc"], ctx["vc"], (seed,))
        (_, amax, _, _), _, _ = _fwd(ctx, parent, tokens)
        lens.add(len(oracle.accept_path(parent, tokens, amax)[1]))
    assert len(lens) >= 3, lens


def test_incremental_levels_equal_one_shot(tiny_ctx):
    """P10: scoring the tree level by level over a growing cache gives bit-identical logits."""
    ctx = tiny_ctx
    parent = gen.tree_branching([4, 2, 1, 1], 16)
    tokens = gen.uniform_tokens(16, ctx["m"].vocab, "cfg1", "tree")
    (full, _, _, _), _, _ = _fwd(ctx, parent, tokens)
    _, _, _, depth = oracle.build_tree_mask(parent, ctx["P"])
    for d in range(int(depth.max()) + 1):
        n = int((depth <= d).sum())
        (part, _, _, _), _, _ = _fwd(ctx, parent[:n], tokens[:n])
        assert np.array_equal(part, full[:n])


def test_relabelling_invariance(tiny_ctx):
    """P11: another topological numbering of the same tree gives the same per-node logits and output."""
    ctx = tiny_ctx
    parent = gen.tree_branching([4, 2, 1, 1], 16)
    tokens = gen.uniform_tokens(16, ctx["m"].vocab, "cfg1", "tree")
    # depth-first preorder numbering
    order = []

    def dfs(n):
        order.append(n)
        for c in np.nonzero(parent == n)[0]:
            dfs(int(c))
    dfs(0)
    order = np.array(order)
    new_id = np.empty(16, np.int64)
    new_id[order] = np.arange(16)
    parent2 = np.array([-1 if parent[o] < 0 else new_id[parent[o]] for o in order], np.int32)
    tokens2 = tokens[order]
    (a, amax_a, _, _), _, _ = _fwd(ctx, parent, tokens)
    (b, amax_b, _, _), _, _ = _fwd(ctx, parent2, tokens2)
    assert np.abs(a[order] - b).max() < 1e-6
    pa, oa = oracle.accept_path(parent, tokens, amax_a)
    pb, ob = oracle.accept_path(parent2, tokens2, amax_b)
    assert list(oa) == list(ob) and list(new_id[pa]) == list(pb)


def test_single_node_tree_is_plain_decoding(tiny_ctx):
    """P12."""
    ctx = tiny_ctx
    rc, mask, pos, depth = oracle.build_tree_mask(np.array([-1], np.int32), ctx["P"])
    assert rc == 0 and int(mask[0, 0]) == 1 and int(mask[0, 1]) == 0 and pos[0] == ctx["P"] and depth[0] == 0
    (logits, amax, _, _), kc, vc = _fwd(ctx, np.array([-1], np.int32), np.array([ctx["root"]], np.int32))
    greedy, gk, gv = oracle_greedy_decode(ctx["cfg"], ctx["nm"], ctx["root"], ctx["P"], ctx["kc"], ctx["vc"], 1)
    assert int(amax[0]) == greedy[0]
    rc, new_len, src, dst = oracle.compact_kv(kc, vc, ctx["P"], np.array([0], np.int32))
    assert new_len == ctx["P"] + 1 and np.array_equal(kc, gk)


def test_cache_rows_hold_bf16_values(tiny_ctx):
    """Contract: K/V rows written by the forward are exactly bf16-representable."""
    ctx = tiny_ctx
    (_, _, _, _), kc, vc = _fwd(ctx, gen.tree_chain(5), gen.uniform_tokens(5, 1024, "c5"))
    rows = kc[:, ctx["P"]:ctx["P"] + 5]
    assert np.array_equal(oracle.from_bf16(oracle.to_bf16(rows)), rows) and np.abs(rows).max() > 0
