"""Small, self-terminating workload for profiler captures: a few verification forwards of a 7B-shaped stack.

    python -m paper_2605_11186_b200.profile_case --layers 2 --tree-size 64 --steps 3

Keeps device memory small (two layers are 0.8 GB of weights, more than the L2) so that a multi-pass
capture of a few launches ends by itself within a minute or two.  Prints the device time per forward.
"""
import argparse

import torch

from . import binding as cats
from . import inputs as gen


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--layers", type=int, default=2)
    ap.add_argument("--tree-size", type=int, default=64)
    ap.add_argument("--prefix", type=int, default=512)
    ap.add_argument("--steps", type=int, default=3)
    ap.add_argument("--model", default="7b", choices=["7b", "13b", "tiny"])
    args = ap.parse_args()
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
