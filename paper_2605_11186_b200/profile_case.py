"""Small, self-terminating workload for profiler captures: a few verification forwards of a 7B-shaped stack.

    python -m paper_2605_11186_b200.profile_case --layers 2 --tree-size 64 --steps 3

Keeps device memory small (two layers are 0.8 GB of weights, more than the L2) so that a multi-pass
capture of a few launches ends by itself within a minute or two.  Prints the device time per forward.
"""
import argparse

import torch

from . import binding as cats
from . import inputs as gen


def attention_only(T, P, steps, nh=32, hd=128):
    import numpy as np
    dev = torch.device("cuda", 0)
    torch.cuda.set_device(dev)
    S, D = P + T, nh * hd
    q = gen.normal_bf16((T, nh, hd), 1.0, dev, "profile", "q")
    k = gen.normal_bf16((S, D), 1.0, dev, "profile", "k")
    v = gen.normal_bf16((S, D), 1.0, dev, "profile", "v")
    parent, _ = gen.tree_topk_shape(T, gen.topk_k_for(T))
    mask = torch.zeros((T, 2), dtype=torch.int64, device=dev)
    pos = torch.zeros(T, dtype=torch.int32, device=dev)
    depth = torch.zeros(T, dtype=torch.int32, device=dev)
    st = cats.new_status()
    cats.cats_build_tree_mask(torch.from_numpy(parent).to(dev), P, mask, pos, depth, st)
    out = torch.zeros((T, nh, hd), dtype=torch.bfloat16, device=dev)
    cfg = cats.model_cfg(gen.ModelShape(hidden=D, n_heads=nh, head_dim=hd, ffn=64, vocab=128, n_layers=1), S)
    ws = cats.new_workspace(cfg, T, P)
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    for i in range(steps):
        e0.record()
        cats.cats_tree_attention(q, k, v, mask, T, P, nh, hd, D, float(1.0 / np.sqrt(hd)), out, ws, st)
        e1.record()
        torch.cuda.synchronize()
        print("attention %d: %.1f us, status %d" % (i, e0.elapsed_time(e1) * 1e3, int(st.item())))


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--layers", type=int, default=2)
    ap.add_argument("--tree-size", type=int, default=64)
    ap.add_argument("--prefix", type=int, default=512)
    ap.add_argument("--steps", type=int, default=3)
    ap.add_argument("--model", default="7b", choices=["7b", "13b", "tiny"])
    ap.add_argument("--attention-only", action="store_true",
                    help="launch only the tree attention of one layer (32 x 128 heads), --steps times, over --prefix cache rows")
    args = ap.parse_args()
    if args.attention_only:
        attention_only(args.tree_size, args.prefix, args.steps)
        return
    shape = {"7b": gen.LLAMA_7B, "13b": gen.LLAMA_13B, "tiny": gen.TINY}[args.model].replace(n_layers=args.layers)
    dev = torch.device("cuda", 0)
    torch.cuda.set_device(dev)
    T, P = args.tree_size, args.prefix
    model = cats.pack_model(gen.make_model(shape, "profile", device=dev), free_source=True)
    kc, vc = gen.make_kv_prefix(shape, args.layers, P + 128, P, "profile", device=dev)
    parent, _ = gen.tree_topk_shape(T, gen.topk_k_for(T))
    tokens = gen.uniform_tokens(T, shape.vocab, "profile", T)
    fwd = cats.VerifyForward(shape, model, kc, vc, T, P, want_logits=False, compact=True)
    d_parent, d_tokens = torch.from_numpy(parent).cuda(), torch.from_numpy(tokens).cuda()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    for i in range(args.steps):
        e0.record()
        fwd.run(d_parent, d_tokens)
        e1.record()
        torch.cuda.synchronize()
        print("forward %d: %.3f ms, %d launches, status %d" % (i, e0.elapsed_time(e1), cats.last_launch_count(),
                                                                int(fwd.status.item())))


if __name__ == "__main__":
    main()
