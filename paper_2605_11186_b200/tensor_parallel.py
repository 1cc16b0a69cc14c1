"""Tensor-parallel tree verification over R GPUs: sharding of a model and the per-rank call sequence.

Rank r holds the attention heads [r*nh/R, (r+1)*nh/R) (rows of Wq/Wk/Wv, columns of Wo, its slice of every K/V cache),
the MLP rows [r*F/R, (r+1)*F/R) (rows of W_gate/W_up, columns of W_down) and the vocabulary rows [r*V/R, (r+1)*V/R) of
the LM head; norm gains, the embedding table and the residual stream are replicated.  Per layer every rank runs the two
half-layer entry points of the library and the ranks sum their [T][hidden] fp32 contributions after each half (an
all-reduce: ``torch.distributed`` over NCCL between GPUs, gloo in the CPU tests of the partition).  Nothing here does
arithmetic on activations: the sums across ranks are the collective's, everything else runs in the library's kernels.

``LocalRanks`` stands in for the process group when all R ranks are emulated one after the other on a single GPU (tests:
the kernels on shard shapes, without a second device); it adds the ranks' contributions with a plain tensor sum.
"""
import numpy as np
import torch

from . import binding as cats


def check_split(shape, R: int) -> None:
    d = shape.n_heads // R * shape.head_dim
    if R < 1 or shape.n_heads % R or shape.ffn % R or shape.vocab % R or d % 64 or (shape.ffn // R) % 8:
        raise ValueError("model shape does not split over %d ranks" % R)


def shard_shape(shape, R: int):
    """The shape one rank's entry points see: full hidden size, 1/R of the heads, the MLP rows and the vocabulary."""
    check_split(shape, R)
    return shape.replace(n_heads=shape.n_heads // R, ffn=shape.ffn // R, vocab=shape.vocab // R)


def shard_layer(w: dict, shape, r: int, R: int) -> dict:
    """Rank r's slices of one layer's nn.Linear matrices ([out][in]); norm gains are replicated."""
    check_split(shape, R)
    d = shape.n_heads // R * shape.head_dim
    f = shape.ffn // R
    rows = slice(r * d, (r + 1) * d)
    frows = slice(r * f, (r + 1) * f)
    return {"attn_norm": w["attn_norm"], "mlp_norm": w["mlp_norm"],
            "wq": w["wq"][rows].contiguous(), "wk": w["wk"][rows].contiguous(), "wv": w["wv"][rows].contiguous(),
            "wo": w["wo"][:, rows].contiguous(),
            "w_gate": w["w_gate"][frows].contiguous(), "w_up": w["w_up"][frows].contiguous(),
            "w_down": w["w_down"][:, frows].contiguous()}


def shard_model(model: dict, shape, r: int, R: int) -> dict:
    v = shape.vocab // R
    return {"shape": shard_shape(shape, R), "layers": [shard_layer(w, shape, r, R) for w in model["layers"]],
            "embed": model["embed"], "final_norm": model["final_norm"], "w_lm": model["w_lm"][r * v:(r + 1) * v].contiguous()}


def shard_cache(cache: torch.Tensor, shape, r: int, R: int) -> torch.Tensor:
    """[layers][max_seq][nh*hd] -> rank r's [layers][max_seq][nh/R*hd]."""
    d = shape.n_heads // R * shape.head_dim
    return cache[:, :, r * d:(r + 1) * d].contiguous()


class LocalRanks:
    """All ranks in this process (one GPU): the collective is a plain sum / stack of the ranks' tensors."""

    def all_reduce(self, tensors):
        total = tensors[0].clone()
        for t in tensors[1:]:
            total += t
        for t in tensors:
            t.copy_(total)

    def all_gather(self, tensors):
        return [torch.stack(tensors) for _ in tensors]


class DistRanks:
    """One rank per process: ``torch.distributed`` (NCCL between GPUs).  Lists hold this process's single tensor."""

    def __init__(self, group=None):
        self.group = group

    def all_reduce(self, tensors):
        torch.distributed.all_reduce(tensors[0], group=self.group)

    def all_gather(self, tensors):
        n = torch.distributed.get_world_size(self.group)
        out = [torch.empty_like(tensors[0]) for _ in range(n)]
        torch.distributed.all_gather(out, tensors[0], group=self.group)
        return [torch.stack(out)]


class _Rank:
    def __init__(self, shape, sshape, model_shard, kcache, vcache, T, prefix_len, r, R, want_logits):
        dev = kcache.device
        self.r = r
        self.cfg = cats.model_cfg(sshape, kcache.shape[1], n_layers=len(model_shard["layers"]))
        self.packed = cats.pack_model(model_shard)
        self.weights = [cats.layer_weights(w) for w in self.packed["layers"]]
        self.kcache, self.vcache = kcache, vcache
        self.ws = cats.new_workspace(self.cfg, T, prefix_len, dev)
        self.status = cats.new_status(dev)
        self.resid = torch.zeros((T, shape.hidden), dtype=torch.float32, device=dev)
        self.partial = torch.zeros((T, shape.hidden), dtype=torch.float32, device=dev)
        self.mask = torch.zeros((T, 2), dtype=torch.int64, device=dev)
        self.pos = torch.zeros(T, dtype=torch.int32, device=dev)
        self.vmax = torch.zeros(T, dtype=torch.float32, device=dev)
        self.vidx = torch.zeros(T, dtype=torch.int32, device=dev)
        self.logits = torch.zeros((T, sshape.vocab), dtype=torch.float32, device=dev) if want_logits else None
        self.argmax = torch.zeros(T, dtype=torch.int32, device=dev)
        self.path = torch.zeros(T, dtype=torch.int32, device=dev)
        self.out_tokens = torch.zeros(T, dtype=torch.int32, device=dev)
        self.scalars = torch.zeros(4, dtype=torch.int32, device=dev)


class TensorParallelVerify:
    """The verification forward split over R ranks.  ``ranks``: the indices this process runs (all of them with
    ``LocalRanks``, one with ``DistRanks``); ``model`` the unsharded nn.Linear-layout model on this process's device,
    ``kcache`` / ``vcache`` the unsharded caches (each rank keeps its head slice)."""

    def __init__(self, shape, model, kcache, vcache, T, prefix_len, R, ranks, comm, want_logits=False):
        self.shape, self.R, self.T, self.P, self.comm = shape, R, T, prefix_len, comm
        self.sshape = shard_shape(shape, R)
        self.ranks = [_Rank(shape, self.sshape, shard_model(model, shape, r, R), shard_cache(kcache, shape, r, R),
                            shard_cache(vcache, shape, r, R), T, prefix_len, r, R, want_logits) for r in ranks]

    def run(self, d_parent, d_tokens, compact=True):
        T, P, shape, ss = self.T, self.P, self.shape, self.sshape
        rk = self.ranks
        for k in rk:
            cats.cats_build_tree_mask(d_parent, P, k.mask, k.pos, None, k.status)
            cats.cats_embed_tokens(k.packed["embed"], d_tokens, k.resid, k.status)
        pending = False
        for l in range(len(rk[0].weights)):
            for k in rk:
                cats.cats_tp_attention_half(k.cfg, k.weights[l], k.resid, k.partial if pending else None, k.kcache[l], k.vcache[l],
                                            k.mask, k.pos, T, P, k.partial, k.ws, k.status)
            self.comm.all_reduce([k.partial for k in rk])
            for k in rk:
                cats.cats_tp_mlp_half(k.cfg, k.weights[l], k.resid, k.partial, T, k.partial, k.ws, k.status)
            self.comm.all_reduce([k.partial for k in rk])
            pending = True
        for k in rk:
            cats.cats_tp_lm_head_shard(k.cfg, k.packed["final_norm"], k.packed["w_lm"], k.resid, k.partial if pending else None, T,
                                       k.r * ss.vocab, k.logits, k.vmax, k.vidx, k.ws, k.status)
        all_max = self.comm.all_gather([k.vmax for k in rk])
        all_idx = self.comm.all_gather([k.vidx for k in rk])
        d = ss.n_heads * ss.head_dim
        for i, k in enumerate(rk):
            cats.cats_tp_argmax_merge(all_max[i].contiguous(), all_idx[i].contiguous(), self.R, T, k.argmax)
            cats.cats_accept_path(d_parent, d_tokens, k.argmax, T, k.path, k.scalars[0:1], k.out_tokens, k.scalars[1:2], k.status)
            if compact:
                L = k.kcache.shape[0]
                cats.cats_compact_kv(k.kcache, k.vcache, L, k.kcache.shape[1] * d, d, P, k.path, k.scalars[0:1], k.scalars[2:3],
                                     None, None, k.status)
        return rk
