"""Tensor-parallel verification on ONE GPU: the R ranks are run one after the other in this process (LocalRanks adds their
contributions where the all-reduce would), so the library's half-layer, vocabulary-shard and merge entry points are
exercised on the shard shapes without a second device and without kernels that wait for one another.  The result must
agree with the oracle's unsplit forward exactly as the single-GPU forward does."""
import numpy as np
import pytest
import torch

import oracle
from paper_2605_11186_b200 import inputs as gen
from helpers import ref_cfg, np_model, cache_to_f32

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def cats():
    from paper_2605_11186_b200 import binding
    assert torch.cuda.is_available()
    return binding


def _case(cats, m, tag, R, parent, P, free_fraction):
    from paper_2605_11186_b200 import tensor_parallel as tp
    T = len(parent)
    max_seq = P + T
    model = gen.make_model(m, tag)
    kc, vc = gen.make_kv_prefix(m, m.n_layers, max_seq, P, tag)
    tokens = gen.uniform_tokens(T, m.vocab, tag, "tokens")
    nm = np_model(model)
    r_k, r_v = cache_to_f32(kc), cache_to_f32(vc)
    logits, amax, margin, _ = oracle.verify_forward(ref_cfg(m, max_seq), nm["layers"], nm["embed"], nm["final_norm"], nm["w_lm"],
                                                    parent, tokens, P, r_k, r_v)
    dmodel = {"layers": [{k: v.cuda() for k, v in w.items()} for w in model["layers"]]}
    for k in ("embed", "final_norm", "w_lm"):
        dmodel[k] = model[k].cuda()
    d_parent, d_tokens = torch.from_numpy(parent).cuda(), torch.from_numpy(tokens).cuda()
    # the unsplit GPU forward, for scale
    base = cats.VerifyForward(m, cats.pack_model(dmodel), kc.cuda(), vc.cuda(), T, P, want_logits=True, compact=True)
    base.run(d_parent, d_tokens)
    torch.cuda.synchronize()
    base_err = float(np.abs(base.logits.cpu().numpy() - logits).max())
    # the split forward, all ranks in this process
    tpv = tp.TensorParallelVerify(m, dmodel, kc.cuda(), vc.cuda(), T, P, R, list(range(R)), tp.LocalRanks(), want_logits=True)
    ranks = tpv.run(d_parent, d_tokens, compact=True)
    torch.cuda.synchronize()
    assert all(int(k.status.item()) == 0 for k in ranks)
    got = torch.cat([k.logits for k in ranks], 1).cpu().numpy()
    err = float(np.abs(got - logits).max())
    print("%s R=%d: split logits err %.4g, unsplit %.4g" % (tag, R, err, base_err))
    assert err <= max(2e-2, free_fraction * base_err + 5e-3)
    g_amax = ranks[0].argmax.cpu().numpy()
    assert all(np.array_equal(k.argmax.cpu().numpy(), g_amax) for k in ranks)          # every rank holds the same merged argmax
    assert np.array_equal(g_amax, got.argmax(-1))                                     # = the argmax of the concatenated shards
    clear = margin > 2 * max(2e-2, err)
    assert np.array_equal(g_amax[clear], amax[clear])
    # walk: bit-exact against the oracle's walk on the same argmax; compaction: a pure move of every rank's slice
    path, out = oracle.accept_path(parent, tokens, g_amax)
    d = m.n_heads // R * m.head_dim
    for k in ranks:
        n = int(k.scalars[0])
        assert np.array_equal(k.path.cpu().numpy()[:n], path) and np.array_equal(k.out_tokens.cpu().numpy()[:int(k.scalars[1])], out)
        assert int(k.scalars[2]) == P + n
    # the ranks' cache slices, side by side, are the unsplit forward's cache (same kernels, other tile shapes: one bf16 ulp)
    k_all = torch.cat([k.kcache for k in ranks], 2).float().cpu().numpy()
    n = len(path)
    ref_rows = base.kcache[:, :P + n].float().cpu().numpy() if np.array_equal(base.path.cpu().numpy()[:int(base.scalars[0])], path) else None
    if ref_rows is not None:
        diff = np.abs(k_all[:, :P + n] - ref_rows)
        mag = np.maximum(np.abs(k_all[:, :P + n]), np.abs(ref_rows))
        assert (diff <= 2.0 ** (np.floor(np.log2(np.maximum(mag, 1e-30))) - 7) * 1.001 + 2e-2).all()
    assert np.array_equal(k_all[:, :P], kc[:, :P].float().numpy())
    return err


def test_tiny_model_two_ranks(cats):
    _case(cats, gen.TINY, "tp_tiny", 2, gen.tree_random(37, 5), 77, 1.5)


def test_7b_shape_two_layers_two_and_four_ranks(cats):
    m = gen.LLAMA_7B.replace(n_layers=2)
    parent, _ = gen.tree_topk_shape(64, 10)
    _case(cats, m, "tp_7b", 2, parent, 512, 1.5)
    _case(cats, m, "tp_7b", 4, parent, 512, 1.5)


WORKER = r'''
import os, sys
sys.path.insert(0, %r)
import numpy as np, torch
from paper_2605_11186_b200 import inputs as gen, binding as cats, tensor_parallel as tp
torch.cuda.set_device(0)
torch.distributed.init_process_group("nccl", device_id=torch.device("cuda", 0))
rank, R = torch.distributed.get_rank(), torch.distributed.get_world_size()
m = gen.TINY
T, P = 16, 64
model = gen.make_model(m, "tp_nccl", device="cuda")
kc, vc = gen.make_kv_prefix(m, m.n_layers, P + T, P, "tp_nccl", device="cuda")
parent = gen.tree_branching([4, 2, 1, 1], T)
tokens = gen.uniform_tokens(T, m.vocab, "tp_nccl", "tokens")
d_parent, d_tokens = torch.from_numpy(parent).cuda(), torch.from_numpy(tokens).cuda()
tpv = tp.TensorParallelVerify(m, model, kc, vc, T, P, R, [rank], tp.DistRanks(), want_logits=True)
k = tpv.run(d_parent, d_tokens)[0]
base = cats.VerifyForward(m, cats.pack_model(model), kc.clone(), vc.clone(), T, P, want_logits=True, compact=True)
base.run(d_parent, d_tokens)
torch.cuda.synchronize()
assert int(k.status.item()) == 0 and int(base.status.item()) == 0
if R == 1:      # one rank holds everything: same kernels on the same shapes, hence the same bits
    assert torch.equal(k.logits, base.logits) and torch.equal(k.argmax, base.argmax) and torch.equal(k.kcache, base.kcache)
print("TP_NCCL_OK", R)
torch.distributed.destroy_process_group()
'''


def test_process_group_path_over_nccl(tmp_path):
    """The torch.distributed path (DistRanks: NCCL all-reduce and all-gather) with the one GPU there is: a world of one
    rank, which must reproduce the unsplit forward bit for bit."""
    import os
    import subprocess
    import sys
    root = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
    script = tmp_path / "tp_nccl_worker.py"
    script.write_text(WORKER % root)
    env = dict(os.environ, MASTER_ADDR="127.0.0.1", NCCL_NVLS_ENABLE="0")
    out = subprocess.run([sys.executable, "-m", "torch.distributed.run", "--nnodes=1", "--nproc-per-node=1", "--master-addr",
                          "127.0.0.1", "--master-port", "29619", str(script)], capture_output=True, text=True, timeout=600, env=env)
    assert out.returncode == 0 and "TP_NCCL_OK 1" in out.stdout, out.stdout[-1500:] + out.stderr[-3000:]
