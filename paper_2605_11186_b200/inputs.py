"""Seeded synthetic inputs: model shapes, random weights, KV prefixes, draft trees.

This module holds none of the method's arithmetic.  It only draws random
numbers and lays out tree shapes; the CUDA path and the CPU oracle are both fed
from the arrays it returns.

Trees are parent arrays in topological order: node 0 is the root (the last
committed token), ``parent[0] == -1`` and ``0 <= parent[i] < i``.
"""
from dataclasses import dataclass, asdict
import zlib

import numpy as np
import torch

MASTER_SEED = 20260511


@dataclass(frozen=True)
class ModelShape:
    hidden: int
    n_heads: int
    head_dim: int
    ffn: int
    vocab: int
    n_layers: int
    rms_eps: float = 1e-5
    rope_base: float = 10000.0

    def replace(self, **kw):
        d = asdict(self)
        d.update(kw)
        return ModelShape(**d)


TINY = ModelShape(hidden=256, n_heads=4, head_dim=64, ffn=688, vocab=1024, n_layers=2)
LLAMA_7B = ModelShape(hidden=4096, n_heads=32, head_dim=128, ffn=11008, vocab=32000, n_layers=32)
LLAMA_13B = ModelShape(hidden=5120, n_heads=40, head_dim=128, ffn=13824, vocab=32000, n_layers=40)

LAYER_MATRICES = ("wq", "wk", "wv", "wo", "w_gate", "w_up", "w_down")
LAYER_NORMS = ("attn_norm", "mlp_norm")


def substream(*key) -> int:
    """A 63-bit seed derived from the master seed and a key such as (config, layer, tensor)."""
    h = zlib.crc32(repr(key).encode())
    h2 = zlib.crc32(repr(key[::-1]).encode(), 0x9E3779B9)
    return (MASTER_SEED * 1000003 + (h << 31) + h2) & 0x7FFFFFFFFFFFFFFF


def _gen(device, *key):
    g = torch.Generator(device=device)
    g.manual_seed(substream(*key))
    return g


def normal_bf16(shape, std, device, *key) -> torch.Tensor:
    """N(0, std) drawn in fp32 from the key's sub-stream, rounded to bf16."""
    g = _gen(device, *key)
    x = torch.empty(shape, dtype=torch.float32, device=device)
    x.normal_(0.0, std, generator=g)
    return x.to(torch.bfloat16)


def layer_shapes(m: ModelShape):
    d = m.n_heads * m.head_dim
    return {"wq": (d, m.hidden), "wk": (d, m.hidden), "wv": (d, m.hidden), "wo": (m.hidden, d),
            "w_gate": (m.ffn, m.hidden), "w_up": (m.ffn, m.hidden), "w_down": (m.hidden, m.ffn)}


def make_layer(m: ModelShape, tag, layer: int, device="cpu", std=0.02) -> dict:
    """One decoder layer: projection matrices N(0, std) in bf16, norm gains 1."""
    w = {}
    for name, shape in layer_shapes(m).items():
        w[name] = normal_bf16(shape, std, device, tag, layer, name)
    for name in LAYER_NORMS:
        w[name] = torch.ones(m.hidden, dtype=torch.bfloat16, device=device)
    return w


def make_model(m: ModelShape, tag, device="cpu", std=0.02, with_head=True, with_embed=True) -> dict:
    model = {"shape": m, "layers": [make_layer(m, tag, l, device, std) for l in range(m.n_layers)]}
    if with_embed:
        model["embed"] = normal_bf16((m.vocab, m.hidden), std, device, tag, "embed")
    if with_head:
        model["final_norm"] = torch.ones(m.hidden, dtype=torch.bfloat16, device=device)
        model["w_lm"] = normal_bf16((m.vocab, m.hidden), std, device, tag, "w_lm")
    return model


def make_kv_prefix(m: ModelShape, n_layers: int, max_seq: int, prefix_len: int, tag, device="cpu"):
    """K and V caches [n_layers, max_seq, n_heads*head_dim] bf16; rows [0, prefix_len) ~ N(0,1), rest 0."""
    d = m.n_heads * m.head_dim
    k = torch.zeros((n_layers, max_seq, d), dtype=torch.bfloat16, device=device)
    v = torch.zeros((n_layers, max_seq, d), dtype=torch.bfloat16, device=device)
    for l in range(n_layers):
        k[l, :prefix_len] = normal_bf16((prefix_len, d), 1.0, device, tag, l, "k_prefix")
        v[l, :prefix_len] = normal_bf16((prefix_len, d), 1.0, device, tag, l, "v_prefix")
    return k, v


def uniform_tokens(n: int, vocab: int, *key) -> np.ndarray:
    rng = np.random.Generator(np.random.Philox(substream(*key)))
    return rng.integers(0, vocab, size=n, dtype=np.int64).astype(np.int32)


def bf16_bits(t: torch.Tensor) -> np.ndarray:
    """Raw bit patterns of a bf16 CPU tensor as a numpy uint16 array (no copy of values' meaning)."""
    assert t.dtype == torch.bfloat16
    return t.detach().cpu().contiguous().view(torch.int16).numpy().view(np.uint16)


# ----------------------------------------------------------------------------
# tree shapes
# ----------------------------------------------------------------------------

def tree_chain(T: int) -> np.ndarray:
    return np.arange(-1, T - 1, dtype=np.int32)


def tree_heap(T: int, arity: int = 4) -> np.ndarray:
    """Balanced ``arity``-ary tree in heap numbering."""
    p = np.empty(T, np.int32)
    p[0] = -1
    for i in range(1, T):
        p[i] = (i - 1) // arity
    return p


def tree_branching(branching, T: int) -> np.ndarray:
    """Every node at depth d gets branching[d] children, numbered breadth-first, cut at T nodes (root included)."""
    parent = [-1]
    level = [0]
    d = 0
    while len(parent) < T and d < len(branching) and level:
        nxt = []
        for n in level:
            for _ in range(branching[d]):
                if len(parent) >= T:
                    break
                parent.append(n)
                nxt.append(len(parent) - 1)
        level = nxt
        d += 1
    if len(parent) != T:
        raise ValueError("branching %r yields only %d nodes, %d asked" % (branching, len(parent), T))
    return np.asarray(parent, np.int32)


def tree_random(T: int, *key, max_children: int = 4) -> np.ndarray:
    """Breadth-first queue; each popped node gets U{1..max_children} children; cut at T nodes."""
    rng = np.random.Generator(np.random.Philox(substream("tree_random", T, *key)))
    parent = [-1]
    queue = [0]
    qi = 0
    while len(parent) < T:
        n = queue[qi]
        qi += 1
        for _ in range(int(rng.integers(1, max_children + 1))):
            if len(parent) >= T:
                break
            parent.append(n)
            queue.append(len(parent) - 1)
    return np.asarray(parent, np.int32)


def topk_fanout(k: int, depth: int, sibling_rank: int) -> int:
    """Fan-out rule of the top-k draft tree: the likeliest child of a shallow node branches widest."""
    return max(1, k >> (depth + sibling_rank))


def tree_topk_shape(T: int, k: int) -> tuple:
    """Shape of a top-k draft tree of T nodes.  Returns (parent, sibling_rank)."""
    parent = [-1]
    rank = [0]
    level = [0]
    d = 0
    while len(parent) < T:
        nxt = []
        for n in level:
            for r in range(topk_fanout(k, d, rank[n])):
                if len(parent) >= T:
                    break
                parent.append(n)
                rank.append(r)
                nxt.append(len(parent) - 1)
        level = nxt
        d += 1
    return np.asarray(parent, np.int32), np.asarray(rank, np.int32)


def tree_cats(gamma: int, correction_positions) -> np.ndarray:
    """CATS-shaped tree: root, a main chain of ``gamma`` draft tokens (nodes 1..gamma), and one leaf
    side branch per position i in ``correction_positions`` (a sibling of main token d_i)."""
    parent = list(range(-1, gamma))
    for i in sorted(correction_positions):
        assert 0 <= i < gamma
        parent.append(i)  # d_i is node i+1, its parent is node i
    return np.asarray(parent, np.int32)


def topk_k_for(T: int) -> int:
    return 4 if T <= 32 else 10
