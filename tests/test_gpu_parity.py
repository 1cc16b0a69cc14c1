"""GPU parity: every C-ABI entry point of libcats against the CPU oracle on the same seeded inputs.

Bit-exact for masks, position ids, paths, tokens and row indices; max-abs-error <= 2e-2 for attention outputs,
the residual stream and the logits; K/V rows within one bf16 ulp.

The contract rounds activations to bf16 at six points per layer, and a rounding is a discontinuity: two valid
evaluations whose fp32/fp64 sums differ in the last bits round a fraction of the activations to neighbouring
bf16 values, and those flips spread through attention and the MLPs.  The oracle measures that spread itself
(fp64- against fp32-accumulated projections, `contract_floor`).  Where the spread of the oracle alone exceeds
2e-2 (7B-shaped layers and short stacks of them) the bound asserted here is 3x that spread instead; test_gpu_stagewise.py
checks every kernel of a layer at the tight tolerance on identical inputs, and test_gpu_full_depth.py checks every layer
of the full-depth 7B / 13B stacks at a flat 2e-2 from the oracle's own inputs (teacher-forced) and reports the
free-running error beside the oracle's drift."""
import numpy as np
import pytest
import torch

import oracle
from paper_2605_11186_b200 import inputs as gen
from helpers import ref_cfg, np_model, np_layer, cache_to_f32, oracle_prefill, planted_tree, assert_bf16_output_close

pytestmark = pytest.mark.gpu

TOL = 2e-2


@pytest.fixture(scope="module")
def cats():
    from paper_2605_11186_b200 import binding
    assert torch.cuda.is_available()
    return binding


def dev(x, dtype=None):
    t = torch.as_tensor(np.ascontiguousarray(x)) if not isinstance(x, torch.Tensor) else x
    if dtype is not None:
        t = t.to(dtype)
    return t.cuda().contiguous()


def dev_layer(w):
    return {k: v.cuda().contiguous() for k, v in w.items()}


def dev_model(model):
    out = {"shape": model["shape"], "layers": [dev_layer(w) for w in model["layers"]]}
    for k in ("embed", "final_norm", "w_lm"):
        if k in model:
            out[k] = model[k].cuda().contiguous()
    return out


def contract_floor(run):
    """run() -> tuple of arrays from the oracle.  Returns (results with fp64 accumulation, max-abs spread per result
    between fp64- and fp32-accumulated projections)."""
    oracle.set_accum32(False)
    a = run()
    oracle.set_accum32(True)
    try:
        b = run()
    finally:
        oracle.set_accum32(False)
    return a, [float(np.abs(np.asarray(x, np.float64) - np.asarray(y, np.float64)).max()) for x, y in zip(a, b)]


def bf16_ulp_close(got_bf16: torch.Tensor, want_f32: np.ndarray):
    """Every element within one bf16 ulp (at the larger magnitude) of the oracle's bf16 value, plus 1e-3 absolute
    for sums that cancel to nearly zero (fp32 accumulation error is absolute, not relative)."""
    g = got_bf16.float().cpu().numpy().astype(np.float64)
    w = want_f32.astype(np.float64)
    mag = np.maximum(np.abs(g), np.abs(w))
    ulp = 2.0 ** (np.floor(np.log2(np.maximum(mag, 1e-30))) - 7)
    bad = np.abs(g - w) > ulp * 1.001 + 1e-3
    return int(bad.sum()), float(np.abs(g - w).max())


ALL_TREES = [
    ("chain1", gen.tree_chain(1)), ("chain16", gen.tree_chain(16)), ("chain128", gen.tree_chain(128)),
    ("b4211", gen.tree_branching([4, 2, 1, 1], 16)), ("b84211", gen.tree_branching([8, 4, 2, 1, 1], 64)),
    ("b632211", gen.tree_branching([6, 3, 2, 2, 1, 1], 64)), ("heap64", gen.tree_heap(64)),
    ("rand128", gen.tree_random(128, 0)), ("rand77", gen.tree_random(77, 1)), ("star100", np.array([-1] + [0] * 99, np.int32)),
    ("topk128", gen.tree_topk_shape(128, 10)[0]), ("topk37", gen.tree_topk_shape(37, 4)[0]),
]


# ---------------------------------------------------------------------------------------------------
# a1: mask / depth / position ids
# ---------------------------------------------------------------------------------------------------

@pytest.mark.parametrize("name,parent", ALL_TREES, ids=[n for n, _ in ALL_TREES])
def test_mask_pos_bit_exact(cats, name, parent):
    T = len(parent)
    P = 1000
    mask = torch.full((T, 2), -1, dtype=torch.int64, device="cuda")
    pos = torch.full((T,), -1, dtype=torch.int32, device="cuda")
    depth = torch.full((T,), -1, dtype=torch.int32, device="cuda")
    st = cats.new_status()
    cats.cats_build_tree_mask(dev(parent), P, mask, pos, depth, st)
    rc, m, p, d = oracle.build_tree_mask(parent, P)
    assert rc == 0 and int(st.item()) == 0
    assert np.array_equal(mask.cpu().numpy().view(np.uint64), m)
    assert np.array_equal(pos.cpu().numpy(), p) and np.array_equal(depth.cpu().numpy(), d)


@pytest.mark.parametrize("parent", [[0, 0, 1], [-1, 1, 0], [-1, 0, 3, 1], [-1, -1], [-1, 0, -5]])
def test_mask_pos_reports_malformed_tree(cats, parent):
    parent = np.array(parent, np.int32)
    T = len(parent)
    mask = torch.full((T + 2, 2), 7, dtype=torch.int64, device="cuda")
    pos = torch.full((T + 2,), 7, dtype=torch.int32, device="cuda")
    st = cats.new_status()
    cats.cats_build_tree_mask(dev(parent), 5, mask, pos, None, st)
    assert int(st.item()) == -2 and oracle.build_tree_mask(parent, 5)[0] == -2
    assert torch.all(mask[:T] == 0) and torch.all(mask[T:] == 7) and torch.all(pos[T:] == 7)   # canaries intact


def test_host_argument_checks(cats):
    st = cats.new_status()
    parent = dev(gen.tree_chain(4))
    mask = torch.zeros((4, 2), dtype=torch.int64, device="cuda")
    pos = torch.zeros(4, dtype=torch.int32, device="cuda")
    with pytest.raises(cats.CatsError) as e:
        cats._check(cats.lib.cats_build_tree_mask(parent.data_ptr(), 129, 0, mask.data_ptr(), pos.data_ptr(), None,
                                                  st.data_ptr(), None), "T=129")
    assert e.value.status == -1
    assert cats.lib.cats_build_tree_mask(None, 4, 0, mask.data_ptr(), pos.data_ptr(), None, st.data_ptr(), None) == -1
    cfg = cats.model_cfg(gen.TINY.replace(head_dim=32), 64)
    assert cats.workspace_bytes(cfg, 16, 64) == 0
    cfg = cats.model_cfg(gen.TINY, 64)
    assert cats.workspace_bytes(cfg, 16, 64) > 0 and cats.workspace_bytes(cfg, 200, 64) == 0


# ---------------------------------------------------------------------------------------------------
# a10: walk, a11: compaction (integer kernels in isolation)
# ---------------------------------------------------------------------------------------------------

def _gpu_walk(cats, parent, tokens, amax):
    T = len(parent)
    path = torch.full((T,), -1, dtype=torch.int32, device="cuda")
    out = torch.full((T,), -1, dtype=torch.int32, device="cuda")
    sc = torch.zeros(2, dtype=torch.int32, device="cuda")
    st = cats.new_status()
    cats.cats_accept_path(dev(parent), dev(tokens), dev(amax), T, path, sc[0:1], out, sc[1:2], st)
    pl, no = [int(v) for v in sc.cpu()]
    assert int(st.item()) == 0
    return path.cpu().numpy()[:pl], out.cpu().numpy()[:no]


@pytest.mark.parametrize("name,parent", ALL_TREES, ids=[n for n, _ in ALL_TREES])
def test_walk_bit_exact(cats, name, parent):
    T = len(parent)
    rng = np.random.default_rng(T)
    for trial in range(6):
        V = [3, 5, 50][trial % 3]
        tokens = rng.integers(0, V, T).astype(np.int32)
        amax = rng.integers(0, V, T).astype(np.int32)
        if trial >= 3:      # plant a long accepted path: follow the first child
            cur = 0
            while True:
                kids = np.nonzero(parent == cur)[0]
                if len(kids) == 0 or rng.random() < 0.1:
                    break
                c = int(kids[rng.integers(0, len(kids))])
                amax[cur] = tokens[c]
                cur = c
        path, out = _gpu_walk(cats, parent, tokens, amax)
        rpath, rout = oracle.accept_path(parent, tokens, amax)
        assert np.array_equal(path, rpath) and np.array_equal(out, rout)


def test_compaction_bit_exact(cats):
    rng = np.random.default_rng(3)
    L, S, R, P = 3, 300, 256, 101
    kc = torch.from_numpy(rng.integers(0, 65535, (L, S, R)).astype(np.int32)).to(torch.int16)
    vc = torch.from_numpy(rng.integers(0, 65535, (L, S, R)).astype(np.int32)).to(torch.int16)
    for path in ([0], [0, 1, 2], [0, 3, 9, 50, 127], [0, 1, 5, 6], list(range(0, 128, 2))):
        path = np.array(path, np.int32)
        dk, dv = kc.cuda(), vc.cuda()
        n = len(path)
        dpath = torch.zeros(128, dtype=torch.int32, device="cuda")
        dpath[:n] = dev(path)
        plen = torch.tensor([n], dtype=torch.int32, device="cuda")
        new_len = torch.zeros(1, dtype=torch.int32, device="cuda")
        src = torch.full((128,), -1, dtype=torch.int32, device="cuda")
        dst = torch.full((128,), -1, dtype=torch.int32, device="cuda")
        st = cats.new_status()
        cats.cats_compact_kv(dk, dv, L, S * R, R, P, dpath, plen, new_len, src, dst, st)
        rk, rv = kc.numpy().copy(), vc.numpy().copy()
        rc, rnew, rsrc, rdst = oracle.compact_kv(rk, rv, P, path)
        assert rc == 0 and int(st.item()) == 0 and int(new_len.item()) == rnew
        assert np.array_equal(src.cpu().numpy()[:n], rsrc) and np.array_equal(dst.cpu().numpy()[:n], rdst)
        assert np.array_equal(dk.cpu().numpy()[:, :rnew], rk[:, :rnew]) and np.array_equal(dv.cpu().numpy()[:, :rnew], rv[:, :rnew])
        assert np.array_equal(dk.cpu().numpy()[:, :P], kc.numpy()[:, :P])
    # a path that is not increasing is reported and nothing moves
    dk, dv = kc.cuda(), vc.cuda()
    dpath = dev(np.array([0, 5, 3], np.int32))
    st = cats.new_status()
    cats.cats_compact_kv(dk, dv, L, S * R, R, P, dpath, torch.tensor([3], dtype=torch.int32, device="cuda"), None, None, None, st)
    assert int(st.item()) == -1 and torch.equal(dk.cpu(), kc)


# ---------------------------------------------------------------------------------------------------
# a5: tree attention alone (config 5 shapes at sizes the oracle finishes quickly, plus ragged cases)
# ---------------------------------------------------------------------------------------------------

CONFIG5_FULL = [(P, name, parent) for P in (256, 1024, 4096, 16384)
                for name, parent in (("chain16", gen.tree_chain(16)), ("heap64", gen.tree_heap(64)), ("rand128", gen.tree_random(128, 5)))]

ATTN_CASES = [
    ("chain16_P256", gen.tree_chain(16), 256, 32, 128), ("heap64_P256", gen.tree_heap(64), 256, 32, 128),
    ("rand128_P256", gen.tree_random(128, 5), 256, 32, 128), ("rand128_P1024", gen.tree_random(128, 5), 1024, 32, 128),
    ("chain16_P1024", gen.tree_chain(16), 1024, 32, 128), ("heap64_P4096", gen.tree_heap(64), 4096, 8, 128),
    ("rand77_P333_hd64", gen.tree_random(77, 2), 333, 4, 64), ("b4211_P128_hd64", gen.tree_branching([4, 2, 1, 1], 16), 128, 4, 64),
    ("chain5_P0", gen.tree_chain(5), 0, 2, 128), ("single_P1", gen.tree_chain(1), 1, 3, 64), ("rand40_P7", gen.tree_random(40, 3), 7, 5, 128),
    ("rand100_P63", gen.tree_random(100, 4), 63, 6, 64),
    # 32 heads, five and seven query tiles: two tiles per CTA with a ragged last group; 49 nodes: the smallest such tree
    ("rand77_P300_h32", gen.tree_random(77, 2), 300, 32, 128), ("rand100_P63_h32", gen.tree_random(100, 4), 63, 32, 128),
    ("rand49_P200_h32", gen.tree_random(49, 6), 200, 32, 128), ("rand48_P200_h32", gen.tree_random(48, 6), 200, 32, 128),
    ("rand128_P896_h32", gen.tree_random(128, 9), 896, 32, 128), ("rand128_P897_h32", gen.tree_random(128, 9), 897, 32, 128),
    # 40 heads: clusters of three CTAs (row blocks of 44, 44 and 40 query rows), and a 17-node tree on them
    ("rand128_P2048_h40", gen.tree_random(128, 11), 2048, 40, 128), ("rand17_P700_h40", gen.tree_random(17, 12), 700, 40, 128),
    # head_dim 64 with 32 heads (the mma.sync kernel): query tiles split over the CTAs of a head, one and two tiles per CTA
    ("heap64_P256_h32_hd64", gen.tree_heap(64), 256, 32, 64), ("rand128_P500_h32_hd64", gen.tree_random(128, 13), 500, 32, 64),
    # shares just below / above the one-block limit of the tcgen05 kernel (192 rows), and a streamed share with a ragged tail
    ("rand33_P735_h32", gen.tree_random(33, 14), 735, 32, 128), ("rand33_P736_h32", gen.tree_random(33, 14), 736, 32, 128),
    ("rand90_P5000_h32", gen.tree_random(90, 15), 5000, 32, 128),
    # no prefix at all; and 140 cache rows over four CTAs of 48 rows each: the last CTA of every cluster has no rows
    ("rand128_P0_h32", gen.tree_random(128, 17), 0, 32, 128), ("rand40_P0_h5", gen.tree_random(40, 18), 0, 5, 128),
    ("rand40_P100_h32", gen.tree_random(40, 16), 100, 32, 128),
]


@pytest.mark.parametrize("name,parent,P,nh,hd", ATTN_CASES, ids=[c[0] for c in ATTN_CASES])
def test_tree_attention_matches_oracle(cats, name, parent, P, nh, hd):
    T = len(parent)
    S = P + T
    D = nh * hd
    q = gen.normal_bf16((T, nh, hd), 1.0, "cpu", "attn", name, "q")
    k = gen.normal_bf16((S + 3, D), 1.0, "cpu", "attn", name, "k")
    v = gen.normal_bf16((S + 3, D), 1.0, "cpu", "attn", name, "v")
    _, mask, _, _ = oracle.build_tree_mask(parent, P)
    scale = 1.0 / np.sqrt(hd)
    want = oracle.tree_attention(q.float().numpy().astype(np.float64), cache_to_f32(k), cache_to_f32(v), mask, P, nh, hd, scale)
    out = torch.zeros((T, nh, hd), dtype=torch.bfloat16, device="cuda")
    cfg = cats.model_cfg(gen.ModelShape(hidden=D, n_heads=nh, head_dim=hd, ffn=64, vocab=128, n_layers=1), S + 3)
    ws = cats.new_workspace(cfg, T, P)
    st = cats.new_status()
    cats.cats_tree_attention(q.cuda(), k.cuda(), v.cuda(), dev(mask.view(np.int64)), T, P, nh, hd, D, float(scale), out, ws, st)
    torch.cuda.synchronize()
    assert int(st.item()) == 0
    assert_bf16_output_close(name, out.float().cpu().numpy(), want, TOL)


@pytest.mark.parametrize("T,P,nh,hd", [(40, 700, 8, 128), (16, 300, 8, 128), (70, 260, 4, 64)])
def test_tree_attention_with_padded_cache_rows(cats, T, P, nh, hd):
    """The cache rows may be wider than n_heads * head_dim (kv_row_stride_elems > n_heads * head_dim): heads are found at
    h * head_dim inside a row, the pad is never read.  The pad is filled with NaN so that a wrong pitch shows."""
    parent = gen.tree_random(T, 21)
    S, D, stride = P + T, nh * hd, nh * hd + 72
    q = gen.normal_bf16((T, nh, hd), 1.0, "cpu", "attn_pad", T, "q")
    k = gen.normal_bf16((S, D), 1.0, "cpu", "attn_pad", T, "k")
    v = gen.normal_bf16((S, D), 1.0, "cpu", "attn_pad", T, "v")
    _, mask, _, _ = oracle.build_tree_mask(parent, P)
    scale = 1.0 / np.sqrt(hd)
    want = oracle.tree_attention(q.float().numpy().astype(np.float64), cache_to_f32(k), cache_to_f32(v), mask, P, nh, hd, scale)
    kw = torch.full((S, stride), float("nan"), dtype=torch.bfloat16, device="cuda")
    vw = torch.full((S, stride), float("nan"), dtype=torch.bfloat16, device="cuda")
    kw[:, :D] = k.cuda()
    vw[:, :D] = v.cuda()
    out = torch.zeros((T, nh, hd), dtype=torch.bfloat16, device="cuda")
    cfg = cats.model_cfg(gen.ModelShape(hidden=D, n_heads=nh, head_dim=hd, ffn=64, vocab=128, n_layers=1), S)
    ws = cats.new_workspace(cfg, T, P)
    st = cats.new_status()
    cats.cats_tree_attention(q.cuda(), kw, vw, dev(mask.view(np.int64)), T, P, nh, hd, stride, float(scale), out, ws, st)
    torch.cuda.synchronize()
    assert int(st.item()) == 0
    g = out.float().cpu().numpy()
    assert np.isfinite(g).all()
    assert_bf16_output_close("padded rows", g, want, TOL)


def _random_attention_shapes(n, seed):
    rng = np.random.default_rng(seed)
    out = []
    for i in range(n):
        T = int(rng.integers(1, 129))
        P = int(rng.choice([0, int(rng.integers(1, 64)), int(rng.integers(64, 700)), int(rng.integers(700, 2600))]))
        nh = int(rng.choice([1, 2, 3, 5, 8, 12, 20, 32, 40]))
        hd = 128 if rng.random() < 0.8 else 64
        out.append((i, T, P, nh, hd))
    return out


@pytest.mark.parametrize("i,T,P,nh,hd", _random_attention_shapes(48, 20260511), ids=lambda v: str(v))
def test_tree_attention_random_shapes(cats, i, T, P, nh, hd):
    """Seeded random shapes: every combination of tree size, prefix length and head count picks its own split of the
    cache rows (cluster size, rows per CTA, one block or streamed, ragged last block); a sample of heads is compared."""
    parent = gen.tree_random(T, 100 + i)
    S, D = P + T, nh * hd
    q = gen.normal_bf16((T, nh, hd), 1.0, "cuda", "attn_rand", i, "q")
    k = gen.normal_bf16((S, D), 1.0, "cuda", "attn_rand", i, "k")
    v = gen.normal_bf16((S, D), 1.0, "cuda", "attn_rand", i, "v")
    _, mask, _, _ = oracle.build_tree_mask(parent, P)
    scale = 1.0 / np.sqrt(hd)
    out = torch.zeros((T, nh, hd), dtype=torch.bfloat16, device="cuda")
    cfg = cats.model_cfg(gen.ModelShape(hidden=D, n_heads=nh, head_dim=hd, ffn=64, vocab=128, n_layers=1), S)
    ws = cats.new_workspace(cfg, T, P)
    st = cats.new_status()
    cats.cats_tree_attention(q, k, v, dev(mask.view(np.int64)), T, P, nh, hd, D, float(scale), out, ws, st)
    torch.cuda.synchronize()
    assert int(st.item()) == 0
    g = out.float().cpu().numpy()
    assert np.isfinite(g).all()
    heads = sorted(set([0, nh - 1, nh // 2]))
    qf, kf, vf = q.float().cpu().numpy().astype(np.float64), k.float().cpu().numpy(), v.float().cpu().numpy()
    for h in heads:
        want = oracle.tree_attention(np.ascontiguousarray(qf[:, h:h + 1]), np.ascontiguousarray(kf[:, h * hd:(h + 1) * hd]),
                                     np.ascontiguousarray(vf[:, h * hd:(h + 1) * hd]), mask, P, 1, hd, scale)
        assert_bf16_output_close("shape %d head %d" % (i, h), g[:, h], want[:, 0], TOL, frac_limit=0.03)


@pytest.mark.parametrize("T,P,nh,hd", [(64, 6000, 32, 128), (128, 3000, 32, 128), (40, 500, 32, 128), (16, 2000, 32, 128), (50, 900, 8, 64)])
def test_tree_attention_is_deterministic(cats, T, P, nh, hd):
    """Same inputs, bit-identical outputs (fixed reduction order), over many launches back to back: the blocks of a share
    are handed between the load, MMA and softmax warps through barriers only, so a missing one would show up here."""
    parent = gen.tree_random(T, 31)
    S, D = P + T, nh * hd
    q = gen.normal_bf16((T, nh, hd), 1.0, "cuda", "attn_det", T, "q")
    k = gen.normal_bf16((S, D), 1.0, "cuda", "attn_det", T, "k")
    v = gen.normal_bf16((S, D), 1.0, "cuda", "attn_det", T, "v")
    _, mask, _, _ = oracle.build_tree_mask(parent, P)
    d_mask = dev(mask.view(np.int64))
    cfg = cats.model_cfg(gen.ModelShape(hidden=D, n_heads=nh, head_dim=hd, ffn=64, vocab=128, n_layers=1), S)
    ws = cats.new_workspace(cfg, T, P)
    st = cats.new_status()
    outs = [torch.zeros((T, nh, hd), dtype=torch.bfloat16, device="cuda") for _ in range(40)]
    for o in outs:
        cats.cats_tree_attention(q, k, v, d_mask, T, P, nh, hd, D, float(1.0 / np.sqrt(hd)), o, ws, st)
    torch.cuda.synchronize()
    assert int(st.item()) == 0
    ref = outs[0].view(torch.int16)
    assert all(torch.equal(o.view(torch.int16), ref) for o in outs[1:])
    assert torch.isfinite(outs[0].float()).all()


@pytest.mark.parametrize("P,name,parent", CONFIG5_FULL, ids=["P%d_%s" % (c[0], c[1]) for c in CONFIG5_FULL])
def test_config5_attention_sweep_full_size(cats, P, name, parent):
    """Config 5 at its full sizes: 32 heads x 128, prefixes up to 16384, the three tree shapes, K/V ~ N(0,1).  The oracle is
    evaluated on a sample of heads (every head is computed independently); all heads of the GPU result are checked for
    finiteness and the sampled ones element by element."""
    T, nh, hd = len(parent), 32, 128
    S, D = P + T, nh * hd
    q = gen.normal_bf16((T, nh, hd), 1.0, "cuda", "cfg5", P, name, "q")
    k = gen.normal_bf16((S, D), 1.0, "cuda", "cfg5", P, name, "k")
    v = gen.normal_bf16((S, D), 1.0, "cuda", "cfg5", P, name, "v")
    _, mask, _, _ = oracle.build_tree_mask(parent, P)
    scale = 1.0 / np.sqrt(hd)
    out = torch.zeros((T, nh, hd), dtype=torch.bfloat16, device="cuda")
    cfg = cats.model_cfg(gen.ModelShape(hidden=D, n_heads=nh, head_dim=hd, ffn=64, vocab=128, n_layers=1), S)
    ws = cats.new_workspace(cfg, T, P)
    st = cats.new_status()
    cats.cats_tree_attention(q, k, v, dev(mask.view(np.int64)), T, P, nh, hd, D, float(scale), out, ws, st)
    torch.cuda.synchronize()
    assert int(st.item()) == 0
    g = out.float().cpu().numpy()
    assert np.isfinite(g).all()
    heads = [0, 13, 31]
    qs = q[:, heads].float().cpu().numpy().astype(np.float64)
    ks = k.view(S, nh, hd)[:, heads].reshape(S, -1).float().cpu().numpy()
    vs = v.view(S, nh, hd)[:, heads].reshape(S, -1).float().cpu().numpy()
    want = oracle.tree_attention(qs, ks, vs, mask, P, len(heads), hd, scale)
    # over 16384 rows the outputs have a standard deviation of about 0.013: the one-ulp bound is the one that bites
    assert_bf16_output_close("P%d %s" % (P, name), g[:, heads], want, TOL)


# ---------------------------------------------------------------------------------------------------
# a3-a8: one decoder layer
# ---------------------------------------------------------------------------------------------------

def _run_layer_case(cats, m, tag, parent, P, resid_std, max_seq):
    T = len(parent)
    w = gen.make_layer(m, tag, 0)
    kc, vc = gen.make_kv_prefix(m, 1, max_seq, P, tag)
    resid = (gen.normal_bf16((T, m.hidden), resid_std, "cpu", tag, "resid").float()
             + 1e-3 * gen.normal_bf16((T, m.hidden), 1.0, "cpu", tag, "resid_lo").float())
    _, mask, pos, _ = oracle.build_tree_mask(parent, P)
    # oracle
    rcfg = ref_cfg(m, max_seq, 1)
    nw = np_layer(w)

    def run():
        r_resid = resid.numpy().copy()
        r_k, r_v = cache_to_f32(kc[0]), cache_to_f32(vc[0])
        oracle.verify_layer(rcfg, nw, r_resid, r_k, r_v, mask, pos, P)
        return r_resid, r_k, r_v
    (r_resid, r_k, r_v), floor = contract_floor(run)
    tol = max(TOL, 3.0 * floor[0])
    # GPU
    cfg = cats.model_cfg(m, max_seq, 1)
    dw = cats.pack_layer(dev_layer(w))
    d_resid = resid.cuda()
    d_k, d_v = kc[0].cuda(), vc[0].cuda()
    ws = cats.new_workspace(cfg, T, P)
    st = cats.new_status()
    cats.cats_verify_layer(cfg, cats.layer_weights(dw), d_resid, d_k, d_v, dev(mask.view(np.int64)), dev(pos), T, P, ws, st)
    torch.cuda.synchronize()
    assert int(st.item()) == 0
    err = np.abs(d_resid.cpu().numpy() - r_resid).max()
    assert err <= tol, (err, tol, floor)
    for got, want in ((d_k, r_k), (d_v, r_v)):
        nbad, maxerr = bf16_ulp_close(got[P:P + T], want[P:P + T])
        assert nbad == 0, (nbad, maxerr)
        assert torch.equal(got[:P].cpu(), (kc if got is d_k else vc)[0, :P])          # prefix untouched
        assert torch.all(got[P + T:] == 0)                                           # nothing written past the tree
    return err


@pytest.mark.parametrize("name,parent", [("b4211", gen.tree_branching([4, 2, 1, 1], 16)), ("rand37", gen.tree_random(37, 7)),
                                         ("chain1", gen.tree_chain(1)), ("rand128", gen.tree_random(128, 8))])
def test_layer_tiny_shape(cats, name, parent):
    """Config-1 layer shape: hidden 256, 4 heads x 64, ffn 688 (ragged tiles), unit-variance hidden states."""
    _run_layer_case(cats, gen.TINY, ("layer_tiny", name), parent, 128, 1.0, 300)


def test_layer_7b_shape(cats):
    """Config 2: one 7B-shaped layer, prefix 1024, 64-node tree [8,4,2,1,1]; embedding-scale and unit-scale inputs."""
    parent = gen.tree_branching([8, 4, 2, 1, 1], 64)
    _run_layer_case(cats, gen.LLAMA_7B, "cfg2", parent, 1024, 0.02, 1024 + 64)
    _run_layer_case(cats, gen.LLAMA_7B, "cfg2_unit", parent, 1024, 1.0, 1024 + 64)


# ---------------------------------------------------------------------------------------------------
# whole forward: config 1 (tiny model, real prefill), 7B- and 13B-shaped stacks
# ---------------------------------------------------------------------------------------------------

def _forward_case(cats, m, tag, parent, tokens, P, max_seq, kc, vc, model, check_compaction=True):
    T = len(parent)
    nm = np_model(model)
    rcfg = ref_cfg(m, max_seq)

    def run():
        r_k, r_v = cache_to_f32(kc), cache_to_f32(vc)
        return oracle.verify_forward(rcfg, nm["layers"], nm["embed"], nm["final_norm"], nm["w_lm"], parent, tokens, P, r_k, r_v)
    (logits, amax, margin, r_resid), floor = contract_floor(run)
    tol = max(TOL, 3.0 * floor[0])
    tol_resid = max(TOL, 3.0 * floor[3])
    dm = cats.pack_model(dev_model(model))
    d_k, d_v = kc.cuda(), vc.cuda()
    fwd = cats.VerifyForward(m, dm, d_k, d_v, T, P, want_logits=True, compact=False)
    fwd.run(dev(parent), dev(tokens))
    torch.cuda.synchronize()
    assert int(fwd.status.item()) == 0
    g_logits = fwd.logits.cpu().numpy()
    err = np.abs(g_logits - logits).max()
    assert err <= tol, (err, tol, floor)
    assert np.abs(fwd.resid.cpu().numpy() - r_resid).max() <= tol_resid
    g_amax = fwd.argmax.cpu().numpy()
    assert np.array_equal(g_amax, g_logits.argmax(-1))               # the GPU's argmax is the argmax of its own logits
    clear = margin > (TOL if tol == TOL else 2 * tol)
    assert np.array_equal(g_amax[clear], amax[clear])
    # walk: integer kernel in isolation, both ways
    g_path = fwd.path.cpu().numpy()[:int(fwd.scalars[0])]
    g_out = fwd.out_tokens.cpu().numpy()[:int(fwd.scalars[1])]
    p2, o2 = oracle.accept_path(parent, tokens, g_amax)
    assert np.array_equal(g_path, p2) and np.array_equal(g_out, o2)
    r_path, r_out = oracle.accept_path(parent, tokens, amax)
    p3, o3 = _gpu_walk(cats, parent, tokens, amax)
    assert np.array_equal(p3, r_path) and np.array_equal(o3, r_out)
    stop_nodes = list(r_path)
    if all(clear[n] for n in stop_nodes):
        assert np.array_equal(g_path, r_path) and np.array_equal(g_out, r_out)
    if check_compaction:
        before_k, before_v = d_k.clone(), d_v.clone()
        new_len = torch.zeros(1, dtype=torch.int32, device="cuda")
        st = cats.new_status()
        L = len(model["layers"])
        D = m.n_heads * m.head_dim
        cats.cats_compact_kv(d_k, d_v, L, max_seq * D, D, P, fwd.path, fwd.scalars[0:1], new_len, None, None, st)
        n = len(g_path)
        assert int(new_len.item()) == P + n and int(st.item()) == 0
        idx = torch.as_tensor(P + g_path, device="cuda", dtype=torch.long)
        assert torch.equal(d_k[:, P:P + n], before_k[:, idx]) and torch.equal(d_v[:, P:P + n], before_v[:, idx])
        assert torch.equal(d_k[:, :P], before_k[:, :P])
    return err, len(g_out)


@pytest.fixture(scope="module")
def cfg1():
    m = gen.TINY
    model = gen.make_model(m, "cfg1")
    P, max_seq = 128, 320
    nm = np_model(model)
    rcfg = ref_cfg(m, max_seq)
    kc = np.zeros((m.n_layers, max_seq, m.n_heads * m.head_dim), np.float32)
    vc = np.zeros_like(kc)
    prompt = gen.uniform_tokens(P, m.vocab, "cfg1", "prompt")
    root = oracle_prefill(rcfg, nm, prompt, kc, vc)
    return dict(m=m, model=model, nm=nm, rcfg=rcfg, kc=kc, vc=vc, P=P, max_seq=max_seq, root=root)


def test_config1_tiny_model(cats, cfg1):
    c = cfg1
    parent = gen.tree_branching([4, 2, 1, 1], 16)
    tokens = gen.uniform_tokens(16, c["m"].vocab, "cfg1", "tree")
    tokens[0] = c["root"]
    kc = torch.from_numpy(c["kc"]).to(torch.bfloat16)
    vc = torch.from_numpy(c["vc"]).to(torch.bfloat16)
    _forward_case(cats, c["m"], "cfg1", parent, tokens, c["P"], c["max_seq"], kc, vc, c["model"])


@pytest.mark.parametrize("T,k,seed", [(16, 4, 0), (16, 4, 1), (32, 4, 2), (40, 10, 3), (128, 10, 4)])
def test_config1_planted_trees_accept_paths(cats, cfg1, T, k, seed):
    """Planted top-k trees: accepted lengths vary, so the walk and compaction move real rows."""
    c = cfg1
    parent, tokens = planted_tree(c["rcfg"], c["nm"], T, k, c["root"], c["P"], c["kc"], c["vc"], (seed,))
    kc = torch.from_numpy(c["kc"]).to(torch.bfloat16)
    vc = torch.from_numpy(c["vc"]).to(torch.bfloat16)
    _forward_case(cats, c["m"], "cfg1", parent, tokens, c["P"], c["max_seq"], kc, vc, c["model"])


def test_fused_forward_with_compaction_and_host_entry(cats, cfg1):
    c = cfg1
    m = c["m"]
    nm = c["nm"]
    # The tiny model's logits are small (std 0.32), so top-1 margins above 2e-2 are rare; its GPU-vs-oracle logit error is
    # below 4e-3 (test_config1_tiny_model reports it), so a path whose margins exceed 1e-2 must come out identical.
    for seed in range(40):
        parent, tokens = planted_tree(c["rcfg"], nm, 16, 4, c["root"], c["P"], c["kc"], c["vc"], (seed,))
        r_k, r_v = c["kc"].copy(), c["vc"].copy()
        _, amax, margin, _ = oracle.verify_forward(c["rcfg"], nm["layers"], nm["embed"], nm["final_norm"], nm["w_lm"], parent,
                                                   tokens, c["P"], r_k, r_v)
        r_path, r_out = oracle.accept_path(parent, tokens, amax)
        if np.all(margin[r_path] > 1e-2) and len(r_path) >= 2:
            break
    else:
        pytest.fail("no planted tree with a clear accepted path")
    dm = cats.pack_model(dev_model(c["model"]))
    kc = torch.from_numpy(c["kc"]).to(torch.bfloat16)
    vc = torch.from_numpy(c["vc"]).to(torch.bfloat16)
    rc, r_new, _, _ = oracle.compact_kv(r_k, r_v, c["P"], r_path)
    d_k, d_v = kc.cuda(), vc.cuda()
    fwd = cats.VerifyForward(m, dm, d_k, d_v, 16, c["P"], want_logits=False, compact=True)
    hp = torch.from_numpy(parent).pin_memory()
    ht = torch.from_numpy(tokens).pin_memory()
    hs = torch.zeros(4, dtype=torch.int32).pin_memory()
    ho = torch.zeros(16, dtype=torch.int32).pin_memory()
    hpath = torch.zeros(16, dtype=torch.int32).pin_memory()
    fwd.run_host(hp, ht, hs, ho, hpath)
    assert list(hs.numpy()) == [len(r_path), len(r_out), r_new, 0]
    assert np.array_equal(ho.numpy()[:len(r_out)], r_out) and np.array_equal(hpath.numpy()[:len(r_path)], r_path)
    nbad, _ = bf16_ulp_close(d_k[0, :r_new], r_k[0, :r_new])      # first layer: only first-stage rounding flips
    assert nbad == 0
    assert np.abs(d_k[:, :r_new].float().cpu().numpy() - r_k[:, :r_new]).max() <= TOL
    assert np.abs(d_v[:, :r_new].float().cpu().numpy() - r_v[:, :r_new]).max() <= TOL


def _stack_case(cats, m, tag, n_layers, parent, P, token_key):
    m = m.replace(n_layers=n_layers)
    T = len(parent)
    max_seq = P + T
    model = gen.make_model(m, tag)
    kc, vc = gen.make_kv_prefix(m, n_layers, max_seq, P, tag)
    tokens = gen.uniform_tokens(T, m.vocab, tag, token_key)
    return _forward_case(cats, m, tag, parent, tokens, P, max_seq, kc, vc, model)


@pytest.mark.parametrize("T,n_layers", [(16, 2), (32, 2), (64, 4), (128, 2)])
def test_7b_shape_stack_with_head(cats, T, n_layers):
    """Config 3 shape (7B layers + LM head, prefix 512, top-k tree shape) on short stacks, every tree size of the sweep."""
    parent, _ = gen.tree_topk_shape(T, gen.topk_k_for(T))
    _stack_case(cats, gen.LLAMA_7B, "cfg3_small", n_layers, parent, 512, T)


def test_13b_shape_layer_stack(cats):
    """Config 4 shape (hidden 5120, 40 heads, ffn 13824, prefix 2048, tree [6,3,2,2,1,1]) on a 2-layer stack."""
    parent = gen.tree_branching([6, 3, 2, 2, 1, 1], 64)
    _stack_case(cats, gen.LLAMA_13B, "cfg4_small", 2, parent, 2048, "t")
