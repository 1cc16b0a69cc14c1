"""Time line of the kernels inside a verification forward (7B-shaped layers, prefix 512).

Builds the measurement variant of the library (``-DCATS_TIMELINE``: the role threads of the projection, attention and
norm kernels store %globaltimer at fixed points, see cats_debug_timeline in include/cats_debug.h), runs a few layers as
one CUDA graph and prints, for one layer in the middle, when each kernel's CTAs entered, saw their dependency resolve,
had their data, and left -- all on one clock, in microseconds after the layer's QKV dependency resolved.

    python -m paper_2605_11186_b200.timeline --tree-size 64

The numbers are a few per cent off the normal build (each stamp is a store), and a launch's CTAs are listed as
min / median / max over the CTAs.  This is how the per-layer budget in the design notes was measured.
"""
import argparse
import os
import sys


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--tree-size", type=int, default=64)
    ap.add_argument("--layers", type=int, default=6)
    ap.add_argument("--prefix", type=int, default=512)
    ap.add_argument("--model", default="7b", choices=["7b", "13b"])
    args = ap.parse_args()

    from . import build
    os.environ["CATS_LIBRARY"] = build.build(timeline=True)
    import numpy as np
    import torch
    from . import binding as cats, inputs as gen

    T, L, P = args.tree_size, args.layers, args.prefix
    shape = (gen.LLAMA_7B if args.model == "7b" else gen.LLAMA_13B).replace(n_layers=L)
    dev = torch.device("cuda", 0)
    model = cats.pack_model(gen.make_model(shape, "timeline", device=dev), free_source=True)
    kc, vc = gen.make_kv_prefix(shape, L, P + 128, P, "timeline", device=dev)
    parent, _ = gen.tree_topk_shape(T, gen.topk_k_for(T))
    tokens = gen.uniform_tokens(T, shape.vocab, "timeline", T)
    fwd = cats.VerifyForward(shape, model, kc, vc, T, P, want_logits=False, compact=True)
    dp, dt = torch.from_numpy(parent).to(dev), torch.from_numpy(tokens).to(dev)
    fwd.run(dp, dt)
    torch.cuda.synchronize()
    g = torch.cuda.CUDAGraph()
    with torch.cuda.graph(g):
        fwd.run(dp, dt)
    for _ in range(3):
        g.replay()
    torch.cuda.synchronize()
    cats.timeline_clear()          # the graph's launches keep their slots; only the stamps are zeroed
    torch.cuda.synchronize()
    g.replay()
    torch.cuda.synchronize()
    assert int(fwd.status.item()) == 0

    def launches(kernel):
        a = cats.timeline(kernel)
        out = [a[i] for i in range(a.shape[0]) if (a[i, :, 0] > 0).any()]
        out.sort(key=lambda s: s[:, 0][s[:, 0] > 0].min())
        return out

    gemm, attn, norm = launches(0), launches(1), launches(2)
    assert len(gemm) == 4 * L + 1 and len(attn) == L, (len(gemm), len(attn), len(norm))
    lay = L // 2                                       # a layer in the middle
    proj = gemm[4 * lay:4 * lay + 5]                   # QKV, O, gate/up, down, next layer's QKV
    t0 = int(np.median(proj[0][:, 4][proj[0][:, 4] > 0]))
    lo, hi = proj[0][:, 0][proj[0][:, 0] > 0].min() - 20000, proj[4][:, 4].max()
    rows = [("QKV", proj[0], GEMM), ("attention", attn[lay], ATTN), ("O", proj[1], GEMM)]
    rows += [("norm", s, NORM) for s in norm if lo < s[:, 0][s[:, 0] > 0].min() < hi]
    rows += [("gate/up", proj[2], GEMM), ("down", proj[3], GEMM), ("QKV (next layer)", proj[4], GEMM)]
    rows.sort(key=lambda r: r[1][:, 0][r[1][:, 0] > 0].min())
    print("time line of layer %d of %d, %s, T=%d, prefix %d (us after the QKV projection's dependency resolved)" % (lay, L, args.model, T, P))
    for name, s, stamps in rows:
        n = int((s[:, 0] > 0).sum())
        print("%s  (%d CTAs)" % (name, n))
        for idx, label in stamps:
            v = s[:, idx]
            v = v[v > 0]
            if len(v):
                v = (v - t0) / 1000.0
                print("    %-32s min %8.2f   median %8.2f   max %8.2f" % (label, v.min(), np.median(v), v.max()))
    period = (np.median(proj[4][:, 4][proj[4][:, 4] > 0]) - t0) / 1000.0
    print("layer period (QKV dependency to the next layer's): %.2f us" % period)


GEMM = [(0, "CTA entered"), (2, "first weight copy issued"), (4, "dependency resolved"), (3, "first stage landed"),
        (6, "last stage landed"), (7, "last accumulator complete"), (8, "epilogue done"), (9, "CTA leaves")]
ATTN = [(0, "CTA entered"), (1, "set-up done"), (2, "dependency resolved"), (4, "Q and first block landed"),
        (6, "first S complete"), (7, "last P written"), (8, "last P V complete"), (9, "records deposited"),
        (10, "records published"), (11, "merged, CTA leaves")]
NORM = [(0, "CTA entered"), (2, "dependency resolved"), (3, "row summed"), (9, "CTA leaves")]

if __name__ == "__main__":
    sys.exit(main())
