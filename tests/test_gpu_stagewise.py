"""Stage-wise GPU parity of one decoder layer: every kernel of the layer is checked against the oracle on the
GPU's own, bit-identical inputs, so no rounding flip of an earlier stage can mask or mimic an error of a later one.

Stages (the library's stage mask stops the layer after each one; the test reads the intermediate buffers out of the
workspace): RMSNorm -> QKV projection + RoPE + KV append -> tree attention -> O projection (+ residual) -> RMSNorm ->
gate/up + SwiGLU -> down projection (+ residual).  bf16 outputs must be within one bf16 ulp of the oracle's value and
differ from it in fewer than 1 % of the elements; fp32 outputs within 1e-3."""
import numpy as np
import pytest
import torch

import oracle
from paper_2605_11186_b200 import inputs as gen
from helpers import np_layer, cache_to_f32

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def cats():
    from paper_2605_11186_b200 import binding
    assert torch.cuda.is_available()
    return binding


def rb(x):
    return oracle.from_bf16(oracle.to_bf16(np.asarray(x, np.float32))).astype(np.float64)


def check_bf16(name, got, want):
    got = np.asarray(got, np.float64)
    want = np.asarray(want, np.float64)
    mag = np.maximum(np.abs(got), np.abs(want))
    ulp = 2.0 ** (np.floor(np.log2(np.maximum(mag, 1e-30))) - 7)
    d = np.abs(got - want)
    bad = d > ulp * 1.001 + 1e-3
    assert not bad.any(), "%s: %d elements off by more than one bf16 ulp, max %g" % (name, int(bad.sum()), d.max())
    frac = float((d > 0).mean())
    assert frac < 0.01, "%s: %.3f %% of the elements differ" % (name, 100 * frac)


def check_f32(name, got, want, tol=1e-3):
    err = float(np.abs(np.asarray(got, np.float64) - np.asarray(want, np.float64)).max())
    assert err <= tol, "%s: max-abs-err %g" % (name, err)


CASES = [
    ("tiny_b4211", gen.TINY, gen.tree_branching([4, 2, 1, 1], 16), 128, 1.0),
    ("tiny_rand37", gen.TINY, gen.tree_random(37, 7), 77, 1.0),
    ("tiny_rand128", gen.TINY, gen.tree_random(128, 8), 100, 1.0),
    ("7b_cfg2", gen.LLAMA_7B, gen.tree_branching([8, 4, 2, 1, 1], 64), 1024, 0.02),
    ("7b_unit_T128", gen.LLAMA_7B, gen.tree_topk_shape(128, 10)[0], 512, 1.0),
    ("13b_cfg4", gen.LLAMA_13B, gen.tree_branching([6, 3, 2, 2, 1, 1], 64), 2048, 1.0),
]


@pytest.mark.parametrize("name,m,parent,P,resid_std", CASES, ids=[c[0] for c in CASES])
def test_layer_stage_by_stage(cats, name, m, parent, P, resid_std):
    T = len(parent)
    max_seq = P + T
    H, nh, hd, F = m.hidden, m.n_heads, m.head_dim, m.ffn
    D = nh * hd
    tag = ("stagewise", name)
    w = gen.make_layer(m, tag, 0)
    # norm gains that are not all one, so that a dropped gain shows
    for n in gen.LAYER_NORMS:
        w[n] = (1.0 + gen.normal_bf16((H,), 0.2, "cpu", tag, n).float()).to(torch.bfloat16)
    nw = np_layer(w)
    kc, vc = gen.make_kv_prefix(m, 1, max_seq, P, tag)
    resid0 = (gen.normal_bf16((T, H), resid_std, "cpu", tag, "resid").float()
              + 1e-3 * gen.normal_bf16((T, H), 1.0, "cpu", tag, "resid_lo").float())
    _, mask, pos, _ = oracle.build_tree_mask(parent, P)

    cfg = cats.model_cfg(m, max_seq, 1)
    packed = cats.pack_layer({k: v.cuda() for k, v in w.items()})    # keep alive: the struct below holds raw pointers
    dw = cats.layer_weights(packed)
    ws = cats.new_workspace(cfg, T, P)
    lay = cats.workspace_layout(cfg, T)
    d_mask = torch.from_numpy(mask.view(np.int64)).cuda()
    d_pos = torch.from_numpy(pos).cuda()

    def run_until(n_stages):
        """Runs the first n_stages stages of the layer from the original inputs; returns (resid, k, v) device tensors."""
        d_resid = resid0.cuda()
        d_k, d_v = kc[0].cuda(), vc[0].cuda()
        st = cats.new_status()
        cats.stage_mask((1 << n_stages) - 1)
        try:
            cats.cats_verify_layer(cfg, dw, d_resid, d_k, d_v, d_mask, d_pos, T, P, ws, st)
            torch.cuda.synchronize()
        finally:
            cats.stage_mask(0x7f)
        assert int(st.item()) == 0
        return d_resid, d_k, d_v

    def act(key, K):
        return cats.unpack_activation(ws[lay[key]:], T, K).float().cpu().numpy().astype(np.float64)

    def parts(n):
        p = ws[lay["part"]:lay["part"] + n * lay["part_stride"] * 4].view(torch.float32).view(n, -1)[:, :T * H]
        return p.view(n, T, H).cpu().numpy().astype(np.float64)

    # stage 0: RMSNorm (the flush at the end of cats_verify_layer folds zero pending partial sums here)
    run_until(1)
    g_xn = act("xn", H)
    check_bf16("xn", g_xn, oracle.rmsnorm(resid0.numpy(), nw["attn_norm"], m.rms_eps))

    # stage 1: QKV + RoPE + KV append, from the GPU's xn
    _, d_k, d_v = run_until(2)
    q = oracle.linear(nw["wq"], g_xn)
    k = oracle.linear(nw["wk"], g_xn)
    v = oracle.linear(nw["wv"], g_xn)
    for t in range(T):
        for h in range(nh):
            q[t, h * hd:(h + 1) * hd] = oracle.rope_head(q[t, h * hd:(h + 1) * hd], int(pos[t]), m.rope_base)
            k[t, h * hd:(h + 1) * hd] = oracle.rope_head(k[t, h * hd:(h + 1) * hd], int(pos[t]), m.rope_base)
    g_q = ws[lay["q"]:lay["q"] + T * D * 2].view(torch.bfloat16).view(T, D).float().cpu().numpy().astype(np.float64)
    g_k = d_k[P:P + T].float().cpu().numpy().astype(np.float64)
    g_v = d_v[P:P + T].float().cpu().numpy().astype(np.float64)
    check_bf16("q", g_q, rb(q))
    check_bf16("k rows", g_k, rb(k))
    check_bf16("v rows", g_v, rb(v))
    assert torch.equal(d_k[:P].cpu(), kc[0, :P]) and torch.equal(d_v[:P].cpu(), vc[0, :P])

    # stage 2: tree attention, from the GPU's q and cache rows
    run_until(3)
    r_k, r_v = cache_to_f32(kc[0]), cache_to_f32(vc[0])
    r_k[P:P + T] = g_k
    r_v[P:P + T] = g_v
    o = oracle.tree_attention(g_q.reshape(T, nh, hd), r_k, r_v, mask, P, nh, hd, 1.0 / np.sqrt(hd)).reshape(T, D)
    g_o = act("o", D)
    check_bf16("attention out", g_o, o)

    # stage 3: O projection; its split-K partial sums are folded by the next RMSNorm: check their sum
    run_until(4)
    wo_out = oracle.linear(nw["wo"], g_o)
    check_f32("o-proj partial sums", parts(lay["pieces_o"]).sum(0), wo_out, 1e-3 * max(1.0, np.abs(wo_out).max()))

    # stage 4: residual add + RMSNorm
    d_resid, _, _ = run_until(5)
    resid1 = (resid0.numpy().astype(np.float64) + wo_out).astype(np.float32)
    g_resid1 = d_resid.cpu().numpy()
    check_f32("resid after attention", g_resid1, resid1, 1e-3 * max(1.0, np.abs(resid1).max()))
    g_xn2 = act("xn", H)
    check_bf16("xn2", g_xn2, oracle.rmsnorm(g_resid1, nw["mlp_norm"], m.rms_eps))

    # stage 5: gate/up + SwiGLU, from the GPU's xn2
    run_until(6)
    g = oracle.linear(nw["w_gate"], g_xn2)
    u = oracle.linear(nw["w_up"], g_xn2)
    g_a = act("act", F)
    check_bf16("swiglu out", g_a, rb(g / (1.0 + np.exp(-g)) * u))

    # stage 6: down projection + residual (the whole layer), from the GPU's SwiGLU output
    d_resid, _, _ = run_until(7)
    down = oracle.linear(nw["w_down"], g_a)
    resid2 = (g_resid1.astype(np.float64) + down).astype(np.float32)
    check_f32("resid after MLP", d_resid.cpu().numpy(), resid2, 1e-3 * max(1.0, np.abs(resid2).max()))


def test_lm_head_from_identical_residual(cats):
    """a9 on identical inputs: final norm + LM head + argmax of a given residual stream, 7B shape, T = 128."""
    m = gen.LLAMA_7B.replace(n_layers=0)
    T = 128
    tag = "lmhead"
    resid = gen.normal_bf16((T, m.hidden), 3.0, "cpu", tag, "resid").float() + 1e-3 * gen.normal_bf16((T, m.hidden), 1.0, "cpu", tag, "lo").float()
    gain = (1.0 + gen.normal_bf16((m.hidden,), 0.2, "cpu", tag, "g").float()).to(torch.bfloat16)
    w_lm = gen.normal_bf16((m.vocab, m.hidden), 0.02, "cpu", tag, "w")
    rcfg = oracle.RefCfg(m.hidden, m.n_heads, m.head_dim, m.ffn, m.vocab, 0, 256, m.rms_eps, m.rope_base)
    logits, amax, margin = oracle.lm_head_argmax(rcfg, gen.bf16_bits(gain), gen.bf16_bits(w_lm), resid.numpy())
    cfg = cats.model_cfg(m, 256, 0)
    ws = cats.new_workspace(cfg, T, 0)
    d_logits = torch.zeros((T, m.vocab), dtype=torch.float32, device="cuda")
    d_amax = torch.zeros(T, dtype=torch.int32, device="cuda")
    st = cats.new_status()
    cats.cats_lm_head_argmax(cfg, gain.cuda(), cats.pack_weights([w_lm.cuda()], 0), resid.cuda(), T, d_logits, d_amax, ws, st)
    torch.cuda.synchronize()
    assert int(st.item()) == 0
    g = d_logits.cpu().numpy()
    assert np.abs(g - logits).max() <= 2e-2
    ga = d_amax.cpu().numpy()
    assert np.array_equal(ga, g.argmax(-1))
    clear = margin > 2e-2
    assert np.array_equal(ga[clear], amax[clear]) and clear.sum() > T // 2
