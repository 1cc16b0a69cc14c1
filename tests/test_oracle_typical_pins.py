"""Pins of the oracle's typical (relaxed) acceptance — the second criterion Acc of Algorithm 1, as the cited Medusa work
defines it: a child token x is acceptable iff p(x) > min(eps, delta * exp(-H(p))), p = softmax(logits / temperature) at
the parent.

What fixes the expected values: torch's logsumexp and Categorical.entropy (library routines), closed forms (uniform and
two-point distributions), the temperature -> 0 limit (the criterion degenerates to greedy acceptance, whose walk is pinned
elsewhere), and Algorithm 1's acceptance loop written out for CATS-shaped trees."""
import math

import numpy as np
import pytest
import torch

import oracle
from paper_2605_11186_b200 import inputs as gen

EPS, DELTA, TEMP = 0.09, 0.3, 0.7


def _rand_logits(rng, T, V, scale=2.0):
    return (rng.standard_normal((T, V)) * scale).astype(np.float32)


def test_stats_match_torch_library_routines():
    rng = np.random.default_rng(0)
    for T, V, t in [(7, 50, 0.7), (16, 1000, 1.0), (3, 32000, 0.3)]:
        parent = gen.tree_random(T, 3)
        tokens = rng.integers(0, V, T).astype(np.int32)
        logits = _rand_logits(rng, T, V, 3.0)
        lse, ent, cand, prob = oracle.typical_stats(logits, t, parent, tokens)
        z = torch.from_numpy(logits).double() / t
        assert np.abs(lse - torch.logsumexp(z, -1).numpy()).max() < 1e-5
        assert np.abs(ent - torch.distributions.Categorical(logits=z).entropy().numpy()).max() < 1e-5
        p = torch.softmax(z, -1).numpy()
        for i in range(1, T):
            assert cand[i] == logits[parent[i], tokens[i]]
            assert abs(prob[i] - p[parent[i], tokens[i]]) < 1e-12
        assert cand[0] == 0 and prob[0] == 0


def test_stats_closed_forms():
    V = 64
    parent = gen.tree_chain(3)
    tokens = np.array([0, 5, 9], np.int32)
    # uniform: H = log V, lse = c/t + log V, p = 1/V
    logits = np.full((3, V), 1.5, np.float32)
    lse, ent, cand, prob = oracle.typical_stats(logits, 0.5, parent, tokens)
    assert np.allclose(ent, math.log(V), atol=1e-6) and np.allclose(lse, 3.0 + math.log(V), atol=1e-6)
    assert np.allclose(prob[1:], 1.0 / V, atol=1e-15)
    # two equal maxima far above the rest: H = log 2, p = 1/2
    logits = np.full((3, V), -1000.0, np.float32)
    logits[:, 5] = logits[:, 9] = 2.0
    lse, ent, cand, prob = oracle.typical_stats(logits, 0.7, parent, tokens)
    assert np.allclose(ent, math.log(2), atol=1e-6) and np.allclose(prob[1:], 0.5, atol=1e-12)
    # one-hot: H = 0, p = 1 at the peak and 0 elsewhere
    logits = np.full((3, V), -1000.0, np.float32)
    logits[:, 5] = 0.0
    lse, ent, cand, prob = oracle.typical_stats(logits, 0.7, parent, tokens)
    assert np.allclose(ent, 0.0, atol=1e-12) and prob[1] == 1.0 and prob[2] == 0.0


def test_uniform_distribution_thresholds():
    """p = 1/V and H = log V: acceptable iff 1/V > min(eps, delta/V).  A wrong sign of H, or max in place of min, fails."""
    V = 40
    parent = gen.tree_branching([2, 2, 1], 9)
    T = len(parent)
    tokens = np.arange(T, dtype=np.int32)
    argmax = np.zeros(T, np.int32)
    logits = np.zeros((T, V), np.float32)
    first_child_chain = [0]
    while True:
        kids = [j for j in range(T) if parent[j] == first_child_chain[-1]]
        if not kids:
            break
        first_child_chain.append(kids[0])
    path, out = oracle.accept_path_typical_def(parent, tokens, argmax, logits, TEMP, EPS, 0.3)
    assert list(path) == first_child_chain and list(out) == [int(tokens[j]) for j in first_child_chain[1:]] + [0]
    path, out = oracle.accept_path_typical_def(parent, tokens, argmax, logits, TEMP, EPS, 2.0)     # 1/V > 2/V is false
    assert list(path) == [0] and list(out) == [0]
    path, _ = oracle.accept_path_typical_def(parent, tokens, argmax, logits, TEMP, 0.001, 2.0)      # 1/V > eps = 0.001
    assert list(path) == first_child_chain


def test_small_temperature_degenerates_to_greedy_walk():
    rng = np.random.default_rng(3)
    checked = 0
    for trial in range(300):
        T = int(rng.integers(2, 40))
        V = 12
        parent = gen.tree_random(T, trial)
        logits = _rand_logits(rng, T, V)
        srt = np.sort(logits, -1)
        if (srt[:, -1] - srt[:, -2]).min() < 0.05:
            continue
        argmax = logits.argmax(-1).astype(np.int32)
        tokens = np.where(rng.random(T) < 0.6, argmax[np.maximum(parent, 0)], rng.integers(0, V, T)).astype(np.int32)
        g_path, g_out = oracle.accept_path(parent, tokens, argmax)
        t_path, t_out = oracle.accept_path_typical_def(parent, tokens, argmax, logits, 1e-3, EPS, DELTA)
        assert list(g_path) == list(t_path) and list(g_out) == list(t_out)
        checked += len(g_path) > 1
    assert checked > 50


def _acc_typical(x, logit_row, t, eps, delta):
    d = torch.distributions.Categorical(logits=torch.from_numpy(logit_row).double() / t)
    return bool(d.probs[x] > min(eps, delta * math.exp(-float(d.entropy()))))


def test_walk_equals_algorithm1_loop_with_typical_acc():
    """Algorithm 1's loop on CATS-shaped trees: at position a the main token d_a is tried first, else the correction at
    that position (judged by the same parent distribution), else stop; bonus = argmax at the last accepted node."""
    rng = np.random.default_rng(5)
    lengths = set()
    took_correction = 0
    for _ in range(1500):
        gamma = int(rng.integers(1, 9))
        corr_pos = sorted(rng.choice(gamma, size=int(rng.integers(0, gamma + 1)), replace=False).tolist())
        parent = gen.tree_cats(gamma, corr_pos)
        T, V = len(parent), 6
        logits = _rand_logits(rng, T, V, 1.5)
        argmax = logits.argmax(-1).astype(np.int32)
        tokens = rng.integers(0, V, T).astype(np.int32)
        corr_node = {i: gamma + 1 + r for r, i in enumerate(corr_pos)}
        nodes, y = [0], []
        for a in range(gamma):
            if _acc_typical(int(tokens[a + 1]), logits[a], TEMP, EPS, DELTA):
                nodes.append(a + 1)
                y.append(int(tokens[a + 1]))
            elif a in corr_node and _acc_typical(int(tokens[corr_node[a]]), logits[a], TEMP, EPS, DELTA):
                nodes.append(corr_node[a])
                y.append(int(tokens[corr_node[a]]))
                took_correction += 1
                break
            else:
                break
        y.append(int(argmax[nodes[-1]]))
        path, out = oracle.accept_path_typical_def(parent, tokens, argmax, logits, TEMP, EPS, DELTA)
        assert list(path) == nodes and list(out) == y
        lengths.add(len(nodes))
    assert len(lengths) >= 5 and took_correction > 20


def test_fp32_log_domain_walk_equals_the_definition():
    """The fixed-precision walk (what the GPU is compared with bit for bit) takes the same decisions as the fp64 definition
    wherever the criterion is not within rounding of its threshold."""
    rng = np.random.default_rng(9)
    inv_t, log_eps, log_delta = np.float32(1.0 / TEMP), np.float32(math.log(EPS)), np.float32(math.log(DELTA))
    n_checked, lengths = 0, set()
    for trial in range(2000):
        T = int(rng.integers(2, 60))
        V = int(rng.integers(4, 30))
        parent = gen.tree_random(T, 1000 + trial)
        logits = _rand_logits(rng, T, V, 1.2)
        argmax = logits.argmax(-1).astype(np.int32)
        tokens = rng.integers(0, V, T).astype(np.int32)
        lse, ent, cand, prob = oracle.typical_stats(logits, TEMP, parent, tokens)
        thr = np.minimum(EPS, DELTA * np.exp(-ent.astype(np.float64)))[np.maximum(parent, 0)]
        if np.abs(np.log(np.maximum(prob[1:], 1e-300)) - np.log(thr[1:])).min() < 1e-4:
            continue
        a = oracle.accept_path_typical_def(parent, tokens, argmax, logits, TEMP, EPS, DELTA)
        b = oracle.accept_path_typical(parent, tokens, argmax, cand, lse, ent, inv_t, log_eps, log_delta)
        assert list(a[0]) == list(b[0]) and list(a[1]) == list(b[1])
        n_checked += 1
        lengths.add(len(a[0]))
    assert n_checked > 1500 and len(lengths) >= 4


def test_typical_accepts_at_least_what_greedy_accepts_when_argmax_is_likely():
    """If the argmax token has p > eps it passes the typical criterion (threshold <= eps): on such inputs the typical
    path is never shorter than the greedy path through the same first-child order."""
    rng = np.random.default_rng(13)
    for trial in range(200):
        gamma = int(rng.integers(1, 10))
        parent = gen.tree_chain(gamma + 1)
        V = 8
        logits = _rand_logits(rng, gamma + 1, V, 2.0)
        argmax = logits.argmax(-1).astype(np.int32)
        tokens = np.concatenate([[0], argmax[:-1]]).astype(np.int32)     # the chain drafts exactly the argmax tokens
        p_top = torch.softmax(torch.from_numpy(logits).double() / TEMP, -1).max(-1).values.numpy()
        if p_top.min() <= EPS:
            continue
        path, out = oracle.accept_path_typical_def(parent, tokens, argmax, logits, TEMP, EPS, DELTA)
        assert list(path) == list(range(gamma + 1)) and list(out[:-1]) == list(tokens[1:])
