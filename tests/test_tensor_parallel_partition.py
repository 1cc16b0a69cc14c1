"""The tensor-parallel partition on CPU: two gloo ranks, each holding half of the heads, of the MLP rows and of the
vocabulary of a tiny model (tensor_parallel.shard_model), evaluate their halves with the ORACLE's primitives, sum their
contributions to the residual stream with an all-reduce after each half layer (where the library's half-layer entry points
put the collective) and merge their (max, index) pairs; the result must equal the oracle's unsplit layer stack and head.

This pins the host logic of the split (which rows and columns a rank holds, where the sums cross ranks, the merge rule of
the vocabulary shards) without a GPU; tests/test_gpu_tensor_parallel.py runs the library's kernels on the shard shapes."""
import json
import os
import subprocess
import sys
import textwrap

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))

WORKER = textwrap.dedent("""
    import os, sys, json
    sys.path.insert(0, %r)
    sys.path.insert(0, os.path.join(%r, "tests"))
    import numpy as np, torch
    import oracle
    from paper_2605_11186_b200 import inputs as gen, tensor_parallel as tp
    from helpers import ref_cfg, np_model, cache_to_f32

    rank = int(os.environ["RANK"]); R = int(os.environ["WORLD_SIZE"])
    torch.distributed.init_process_group("gloo")
    comm = tp.DistRanks()
    m = gen.TINY
    T, P, max_seq = 21, 40, 80
    model = gen.make_model(m, "tp_cpu")
    kc, vc = gen.make_kv_prefix(m, m.n_layers, max_seq, P, "tp_cpu")
    parent = gen.tree_random(T, 3)
    tokens = gen.uniform_tokens(T, m.vocab, "tp_cpu", "tokens")
    _, mask, pos, _ = oracle.build_tree_mask(parent, P)

    # ---- this rank's shard, evaluated with the oracle's primitives ----
    ss = tp.shard_shape(m, R)
    sm = np_model(tp.shard_model(model, m, rank, R))
    s_k, s_v = cache_to_f32(tp.shard_cache(kc, m, rank, R)), cache_to_f32(tp.shard_cache(vc, m, rank, R))
    nh, hd = ss.n_heads, ss.head_dim
    D = nh * hd

    def rnd(x):
        return oracle.from_bf16(oracle.to_bf16(np.asarray(x, np.float32))).astype(np.float64)

    def all_reduce(x):
        t = torch.from_numpy(np.ascontiguousarray(x))
        comm.all_reduce([t])
        return t.numpy()

    resid = oracle.embed(sm["embed"], tokens)
    for l in range(m.n_layers):
        w = sm["layers"][l]
        xn = oracle.rmsnorm(resid, w["attn_norm"], m.rms_eps)
        q, k, v = oracle.linear(w["wq"], xn), oracle.linear(w["wk"], xn), oracle.linear(w["wv"], xn)
        for t in range(T):
            for h in range(nh):
                q[t, h * hd:(h + 1) * hd] = oracle.rope_head(q[t, h * hd:(h + 1) * hd], int(pos[t]), m.rope_base)
                k[t, h * hd:(h + 1) * hd] = oracle.rope_head(k[t, h * hd:(h + 1) * hd], int(pos[t]), m.rope_base)
        s_k[l, P:P + T] = rnd(k)
        s_v[l, P:P + T] = rnd(v)
        o = oracle.tree_attention(rnd(q).reshape(T, nh, hd), s_k[l], s_v[l], mask, P, nh, hd, 1.0 / np.sqrt(hd))
        c1 = all_reduce(oracle.linear(w["wo"], o.reshape(T, D)))                  # the sum over ranks = Wo . o
        resid = (resid.astype(np.float64) + c1).astype(np.float32)
        xn = oracle.rmsnorm(resid, w["mlp_norm"], m.rms_eps)
        g, u = oracle.linear(w["w_gate"], xn), oracle.linear(w["w_up"], xn)
        a = rnd(g / (1.0 + np.exp(-g)) * u)
        c2 = all_reduce(oracle.linear(w["w_down"], a))
        resid = (resid.astype(np.float64) + c2).astype(np.float32)
    logits = oracle.linear(sm["w_lm"], oracle.rmsnorm(resid, sm["final_norm"], m.rms_eps)).astype(np.float32)
    vmax = torch.from_numpy(logits.max(-1).copy())
    vidx = torch.from_numpy((logits.argmax(-1) + rank * ss.vocab).astype(np.int32))
    all_max = comm.all_gather([vmax])[0].numpy()
    all_idx = comm.all_gather([vidx])[0].numpy()
    best = all_max.max(0)
    amax = np.array([min(all_idx[r, t] for r in range(R) if all_max[r, t] == best[t]) for t in range(T)], np.int32)

    # ---- the unsplit oracle ----
    nm = np_model(model)
    r_k, r_v = cache_to_f32(kc), cache_to_f32(vc)
    full_logits, full_amax, margin, full_resid = oracle.verify_forward(ref_cfg(m, max_seq), nm["layers"], nm["embed"], nm["final_norm"],
                                                                      nm["w_lm"], parent, tokens, P, r_k, r_v)
    d0 = rank * D
    out = {"rank": rank,
           "resid_err": float(np.abs(resid - full_resid).max()),
           "logits_err": float(np.abs(logits - full_logits[:, rank * ss.vocab:(rank + 1) * ss.vocab]).max()),
           "cache_err": float(max(np.abs(s_k - r_k[:, :, d0:d0 + D]).max(), np.abs(s_v - r_v[:, :, d0:d0 + D]).max())),
           "argmax_equal": bool(np.array_equal(amax[margin > 1e-4], full_amax[margin > 1e-4]))}
    print("RESULT " + json.dumps(out), flush=True)
    torch.distributed.barrier()
    torch.distributed.destroy_process_group()
""") % (ROOT, ROOT)


def test_two_ranks_reproduce_the_unsplit_oracle(tmp_path):
    script = tmp_path / "tp_worker.py"
    script.write_text(WORKER)
    env = dict(os.environ, MASTER_ADDR="127.0.0.1", OMP_NUM_THREADS="2")
    out = subprocess.run([sys.executable, "-m", "torch.distributed.run", "--nnodes=1", "--nproc-per-node=2",
                          "--master-addr", "127.0.0.1", "--master-port", "29617", str(script)],
                         capture_output=True, text=True, timeout=600, env=env)
    assert out.returncode == 0, out.stdout[-1500:] + out.stderr[-3000:]
    import re
    res = [json.loads(x) for x in re.findall(r"RESULT (\{[^{}]*\})", out.stdout)]       # the two ranks may share a line
    assert sorted(r["rank"] for r in res) == [0, 1]
    for r in res:
        # the split only reorders fp64 sums (1e-15); the fp32 residual stream and the bf16 rounding points turn that into
        # a few flips of the last bit
        assert r["resid_err"] < 2e-3 and r["logits_err"] < 2e-3 and r["cache_err"] < 1e-2, r
        assert r["argmax_equal"], r


def test_shard_shapes_and_slices():
    sys.path.insert(0, ROOT)
    import pytest
    import torch
    from paper_2605_11186_b200 import inputs as gen, tensor_parallel as tp
    m = gen.LLAMA_7B
    s = tp.shard_shape(m, 4)
    assert (s.hidden, s.n_heads, s.ffn, s.vocab) == (4096, 8, 2752, 8000)
    with pytest.raises(ValueError):
        tp.shard_shape(m, 3)                    # 32 heads do not split in three
    with pytest.raises(ValueError):
        tp.shard_shape(gen.TINY, 4)             # one head of 64 per rank: fine; 688 / 4 = 172 is not a multiple of 8
    t = gen.TINY
    w = {k: torch.arange(a * b, dtype=torch.float32).reshape(a, b) for k, (a, b) in gen.layer_shapes(t).items()}
    w["attn_norm"] = w["mlp_norm"] = torch.ones(t.hidden)
    parts = [tp.shard_layer(w, t, r, 2) for r in range(2)]
    assert torch.equal(torch.cat([p["wq"] for p in parts], 0), w["wq"])
    assert torch.equal(torch.cat([p["wo"] for p in parts], 1), w["wo"])
    assert torch.equal(torch.cat([p["w_up"] for p in parts], 0), w["w_up"])
    assert torch.equal(torch.cat([p["w_down"] for p in parts], 1), w["w_down"])
