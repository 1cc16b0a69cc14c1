"""Shared test helpers: conversions between the input generators' torch tensors and the oracle's
numpy arrays, oracle-driven prefill, and the planted top-k draft tree (built with the oracle only)."""
import numpy as np
import torch

import oracle
from paper_2605_11186_b200 import inputs as gen


def ref_cfg(m: gen.ModelShape, max_seq: int, n_layers=None) -> oracle.RefCfg:
    return oracle.RefCfg(m.hidden, m.n_heads, m.head_dim, m.ffn, m.vocab,
                         m.n_layers if n_layers is None else n_layers, max_seq, m.rms_eps, m.rope_base)


def np_layer(w: dict) -> dict:
    return {k: gen.bf16_bits(v) for k, v in w.items()}


def np_model(model: dict) -> dict:
    out = {"shape": model["shape"], "layers": [np_layer(w) for w in model["layers"]]}
    for k in ("embed", "final_norm", "w_lm"):
        if k in model:
            out[k] = gen.bf16_bits(model[k])
    return out


def cache_to_f32(t: torch.Tensor) -> np.ndarray:
    """bf16 torch cache -> float32 numpy (exact)."""
    return t.detach().cpu().to(torch.float32).numpy().copy()


def oracle_prefill(cfg, nm, prompt_tokens, kc, vc):
    """Fill cache rows [0, len(prompt)) by running the oracle over the prompt as chain trees of <=128
    nodes.  Returns the argmax at the last prompt position (the first generated token)."""
    P = 0
    amax = None
    prompt_tokens = np.asarray(prompt_tokens, np.int32)
    while P < len(prompt_tokens):
        n = min(128, len(prompt_tokens) - P)
        parent = gen.tree_chain(n)
        _, amax, _, _ = oracle.verify_forward(cfg, nm["layers"], nm["embed"], nm["final_norm"], nm["w_lm"],
                                              parent, prompt_tokens[P:P + n], P, kc, vc, want_logits=False)
        P += n
    return int(amax[-1])


def oracle_greedy_decode(cfg, nm, first_token, P, kc, vc, n_steps):
    """Ordinary token-by-token greedy decoding with the oracle (T=1 trees).  kc/vc are copied."""
    kc = kc.copy()
    vc = vc.copy()
    toks = []
    cur = int(first_token)
    for s in range(n_steps):
        _, amax, _, _ = oracle.verify_forward(cfg, nm["layers"], nm["embed"], nm["final_norm"], nm["w_lm"],
                                              np.array([-1], np.int32), np.array([cur], np.int32), P + s, kc, vc,
                                              want_logits=False)
        cur = int(amax[0])
        toks.append(cur)
    return toks, kc, vc


def planted_tree(cfg, nm, T, k, root_token, P, kc, vc, seed_key, p_keep=0.7):
    """Top-k draft tree whose child tokens are taken from the oracle's own top-k logits at each node.

    Built level by level: the oracle scores the nodes placed so far, then each node of the deepest level
    gets ``topk_fanout`` children carrying its rank-0..f-1 tokens (with probability p_keep) or ranks 1..f
    (top-1 withheld).  Returns (parent, tokens)."""
    parent_full, rank = gen.tree_topk_shape(T, k)
    rng = np.random.Generator(np.random.Philox(gen.substream("planted", T, k, *seed_key)))
    _, _, _, depth = oracle.build_tree_mask(parent_full, P)
    tokens = np.zeros(T, np.int32)
    tokens[0] = root_token
    maxd = int(depth.max())
    for d in range(maxd):
        n_have = int(np.sum(depth <= d))
        kcc, vcc = kc.copy(), vc.copy()
        logits, _, _, _ = oracle.verify_forward(cfg, nm["layers"], nm["embed"], nm["final_norm"], nm["w_lm"],
                                                parent_full[:n_have], tokens[:n_have], P, kcc, vcc)
        for n in np.nonzero(depth == d)[0]:
            kids = np.nonzero(parent_full == n)[0]
            if len(kids) == 0:
                continue
            order = np.argsort(-logits[n], kind="stable")
            keep = rng.random() < p_keep
            start = 0 if keep else 1
            for r, c in enumerate(kids):
                tokens[c] = order[start + r]
    return parent_full, tokens


def assert_bf16_output_close(name, got, want, tol, frac_limit=0.02):
    """A bf16 output against the oracle's values: the stated absolute tolerance, and -- the bound that still bites
    when the values themselves are small, as attention outputs over long prefixes are -- every element within one
    bf16 ulp (at the larger magnitude) plus 1e-3 of the largest expected value, and only a small fraction of the
    elements differing at all.  Returns (max-abs-err, max |want|) for the caller's report."""
    g = np.asarray(got, np.float64)
    w = np.asarray(want, np.float64)
    wmax = float(np.abs(w).max())
    d = np.abs(g - w)
    err = float(d.max())
    assert err <= tol, "%s: max-abs-err %g > %g (max |want| %g)" % (name, err, tol, wmax)
    wb = w.astype(np.float32).astype(np.float64)
    mag = np.maximum(np.abs(g), np.abs(wb))
    ulp = 2.0 ** (np.floor(np.log2(np.maximum(mag, 1e-30))) - 7)
    bad = d > ulp * 1.001 + 1e-3 * wmax
    assert not bad.any(), "%s: %d elements off by more than one bf16 ulp, max-abs-err %g, max |want| %g" % (
        name, int(bad.sum()), err, wmax)
    # elements that differ from the oracle's value rounded to bf16
    import torch
    w16 = torch.from_numpy(w.astype(np.float32)).to(torch.bfloat16).float().numpy().astype(np.float64)
    frac = float((g != w16).mean())
    assert frac < frac_limit, "%s: %.2f %% of the elements differ from the rounded oracle value" % (name, 100 * frac)
    print("%s: max-abs-err %.3g, max |want| %.3g, %.2f %% of elements differ" % (name, err, wmax, 100 * frac))
    return err, wmax
