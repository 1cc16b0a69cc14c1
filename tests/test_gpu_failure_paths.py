"""Failure paths of libcats on the GPU: bounded device-side waits that run out, and host-visible argument errors.

No GPU fault is provoked anywhere.  A wait is made to run out on the host's initiative: the library's fault-injection
hook withholds one signal (a ready flag of the projection kernel, the query copy of the attention kernel) and the wait
limit is shortened to 2 ms, so the waiting threads give up, the kernel reports CATS_ERR_TIMEOUT through the status word
and returns normally.  The tests then check that nothing was written outside the output buffers and that the next,
undisturbed call on the same workspace gives the undisturbed result bit for bit (no flag or barrier state is left
behind)."""
import numpy as np
import pytest
import torch

import oracle
from paper_2605_11186_b200 import inputs as gen

pytestmark = pytest.mark.gpu

TIMEOUT = -6
GUARD = 64


@pytest.fixture(scope="module")
def cats():
    from paper_2605_11186_b200 import binding
    assert torch.cuda.is_available()
    return binding


@pytest.fixture()
def short_waits(cats):
    cats.wait_limit_ns(2_000_000)
    try:
        yield
    finally:
        cats.inject_fault(0)
        cats.wait_limit_ns(0)


def _layer_setup(cats, tag):
    m = gen.TINY
    parent = gen.tree_random(37, 7)
    T, P, max_seq = len(parent), 77, 160
    w = gen.make_layer(m, tag, 0)
    kc, vc = gen.make_kv_prefix(m, 1, max_seq, P, tag)
    resid = gen.normal_bf16((T, m.hidden), 1.0, "cpu", tag, "resid").float()
    _, mask, pos, _ = oracle.build_tree_mask(parent, P)
    cfg = cats.model_cfg(m, max_seq, 1)
    packed = cats.pack_layer({k: v.cuda() for k, v in w.items()})
    return dict(m=m, T=T, P=P, max_seq=max_seq, cfg=cfg, packed=packed, lw=cats.layer_weights(packed), kc=kc, vc=vc, resid=resid,
                mask=torch.from_numpy(mask.view(np.int64)).cuda(), pos=torch.from_numpy(pos).cuda())


def _run_layer(cats, s, ws):
    """One cats_verify_layer call on guarded buffers.  Returns (status, resid, kcache, vcache, guards_intact)."""
    T, H = s["T"], s["m"].hidden
    resid = torch.full((T + 2 * GUARD, H), 7.0, dtype=torch.float32, device="cuda")
    resid[GUARD:GUARD + T] = s["resid"].cuda()
    d_k, d_v = s["kc"][0].cuda(), s["vc"][0].cuda()
    st = cats.new_status()
    cats.cats_verify_layer(s["cfg"], s["lw"], resid[GUARD:GUARD + T], d_k, d_v, s["mask"], s["pos"], T, s["P"], ws, st)
    torch.cuda.synchronize()
    intact = bool(torch.all(resid[:GUARD] == 7.0)) and bool(torch.all(resid[GUARD + T:] == 7.0)) and \
        bool(torch.all(d_k[s["P"] + T:] == 0)) and bool(torch.all(d_v[s["P"] + T:] == 0)) and \
        torch.equal(d_k[:s["P"]].cpu(), s["kc"][0, :s["P"]]) and torch.equal(d_v[:s["P"]].cpu(), s["vc"][0, :s["P"]])
    return int(st.item()), resid[GUARD:GUARD + T].clone(), d_k, d_v, intact


def test_projection_flag_wait_runs_out_and_the_next_call_is_clean(cats, short_waits):
    """Tiny-model layer: its QKV and gate/up projections have tiles shared between CTAs, finished by the tile's owner once
    the contributors' flags are up.  With the flags withheld every owner's wait runs out."""
    s = _layer_setup(cats, "fail_gemm")
    ws = cats.new_workspace(s["cfg"], s["T"], s["P"])
    st0, want_resid, want_k, want_v, ok0 = _run_layer(cats, s, ws)
    assert st0 == 0 and ok0
    cats.inject_fault(1)
    st1, _, _, _, ok1 = _run_layer(cats, s, ws)
    assert st1 == TIMEOUT, st1                    # reported, not trapped: the context is alive and the call returned
    assert ok1                                    # nothing outside the outputs was touched
    cats.inject_fault(0)
    st2, got_resid, got_k, got_v, ok2 = _run_layer(cats, s, ws)     # same workspace, no clean-up by the caller
    assert st2 == 0 and ok2
    assert torch.equal(got_resid, want_resid) and torch.equal(got_k, want_k) and torch.equal(got_v, want_v)


def test_attention_barrier_wait_runs_out_and_the_next_call_is_clean(cats, short_waits):
    """tcgen05 attention (head_dim 128), clusters of several CTAs, one-block and streamed shares: the query tile is
    announced on its barrier but never copied, so the thread that issues Q K^T gives up, and with it the CTA."""
    for T, P, nh in ((40, 700, 8), (64, 512, 32), (33, 6000, 32)):
        hd = 128
        parent = gen.tree_random(T, 5)
        S, D = P + T, nh * hd
        q = gen.normal_bf16((T, nh, hd), 1.0, "cuda", "fail_attn", T, "q")
        k = gen.normal_bf16((S, D), 1.0, "cuda", "fail_attn", T, "k")
        v = gen.normal_bf16((S, D), 1.0, "cuda", "fail_attn", T, "v")
        _, mask, _, _ = oracle.build_tree_mask(parent, P)
        d_mask = torch.from_numpy(mask.view(np.int64)).cuda()
        cfg = cats.model_cfg(gen.ModelShape(hidden=D, n_heads=nh, head_dim=hd, ffn=64, vocab=128, n_layers=1), S)
        ws = cats.new_workspace(cfg, T, P)

        def run():
            out = torch.full((T + 2 * GUARD, nh, hd), 3.0, dtype=torch.bfloat16, device="cuda")
            st = cats.new_status()
            cats.cats_tree_attention(q, k, v, d_mask, T, P, nh, hd, D, float(1.0 / np.sqrt(hd)), out[GUARD:GUARD + T], ws, st)
            torch.cuda.synchronize()
            intact = bool(torch.all(out[:GUARD] == 3.0)) and bool(torch.all(out[GUARD + T:] == 3.0))
            return int(st.item()), out[GUARD:GUARD + T].clone(), intact
        st0, want, ok0 = run()
        assert st0 == 0 and ok0
        cats.inject_fault(2)
        st1, _, ok1 = run()
        cats.inject_fault(0)
        assert st1 == TIMEOUT and ok1, (T, P, nh, st1)
        st2, got, ok2 = run()
        assert st2 == 0 and ok2 and torch.equal(got.view(torch.int16), want.view(torch.int16)), (T, P, nh)


def test_walk_stays_in_bounds_on_a_malformed_parent_array(cats):
    """A parent array with a cycle through the root whose tokens all match the argmax: the walk must neither run past
    its T-entry outputs nor loop; it reports CATS_ERR_BAD_TREE."""
    for parent in ([0, 0, 1, 2], [3, 0, 1, 2], [-1, 2, 1, 0]):
        T = len(parent)
        d_parent = torch.tensor(parent, dtype=torch.int32, device="cuda")
        tokens = torch.full((T,), 5, dtype=torch.int32, device="cuda")
        amax = torch.full((T,), 5, dtype=torch.int32, device="cuda")
        path = torch.full((T + GUARD,), -9, dtype=torch.int32, device="cuda")
        out = torch.full((T + GUARD,), -9, dtype=torch.int32, device="cuda")
        sc = torch.zeros(2, dtype=torch.int32, device="cuda")
        st = cats.new_status()
        cats.cats_accept_path(d_parent, tokens, amax, T, path[:T], sc[0:1], out[:T], sc[1:2], st)
        torch.cuda.synchronize()
        assert int(st.item()) == -2
        assert torch.all(path[T:] == -9) and torch.all(out[T:] == -9)
        n = int(sc[0])
        assert 1 <= n <= T and int(sc[1]) == n
        p = path[:n].cpu().numpy()
        assert p[0] == 0 and np.all(np.diff(p) > 0)


def test_forward_reports_a_malformed_tree_and_stays_in_bounds(cats):
    m = gen.TINY
    T, P, max_seq = 8, 16, 64
    model = gen.make_model(m, "fail_fwd")
    dm = {"layers": [{k: v.cuda() for k, v in w.items()} for w in model["layers"]]}
    for k in ("embed", "final_norm", "w_lm"):
        dm[k] = model[k].cuda()
    dm = cats.pack_model(dm)
    kc, vc = gen.make_kv_prefix(m, m.n_layers, max_seq, P, "fail_fwd")
    fwd = cats.VerifyForward(m, dm, kc.cuda(), vc.cuda(), T, P, want_logits=False, compact=True)
    parent = torch.tensor([0, 0, 1, 2, 3, 4, 5, 6], dtype=torch.int32, device="cuda")     # parent[0] must be -1
    tokens = torch.zeros(T, dtype=torch.int32, device="cuda")
    fwd.run(parent, tokens)
    torch.cuda.synchronize()
    assert int(fwd.status.item()) == -2
    assert 1 <= int(fwd.scalars[0]) <= T


def test_host_visible_errors_launch_nothing(cats):
    s = _layer_setup(cats, "fail_host")
    T, P, H = s["T"], s["P"], s["m"].hidden
    ws = cats.new_workspace(s["cfg"], T, P)
    resid = s["resid"].cuda()
    before = resid.clone()
    d_k, d_v = s["kc"][0].cuda(), s["vc"][0].cuda()
    st = cats.new_status()

    def layer(**kw):
        a = dict(cfg=s["cfg"], w=s["lw"], resid=resid, k=d_k, v=d_v, mask=s["mask"], pos=s["pos"], T=T, P=P, ws=ws)
        a.update(kw)
        cats.cats_verify_layer(a["cfg"], a["w"], a["resid"], a["k"], a["v"], a["mask"], a["pos"], a["T"], a["P"], a["ws"], st)

    def refused(code, **kw):
        with pytest.raises(cats.CatsError) as e:
            layer(**kw)
        assert e.value.status == code, (kw.keys(), e.value.status)
        assert cats.last_launch_count() == 0
    refused(-4, ws=ws[:-1])                                          # one byte short
    refused(-4, ws=ws[8:])                                           # not 1024-byte aligned
    refused(-1, resid=resid.view(-1)[1:1 + (T - 1) * H].view(T - 1, H), T=T - 1)    # residual not 16-byte aligned
    refused(-1, P=s["max_seq"] - T + 1)                              # prefix_len + T > max_seq
    refused(-1, T=129)
    refused(-1, T=0)
    bad_cfg = cats.model_cfg(s["m"].replace(head_dim=96), s["max_seq"], 1)
    refused(-3, cfg=bad_cfg)
    # LM head and attention: short workspace
    model = gen.make_model(s["m"], "fail_host")
    dm = cats.pack_model({"layers": [], "embed": model["embed"].cuda(), "final_norm": model["final_norm"].cuda(),
                          "w_lm": model["w_lm"].cuda()})
    amax = torch.zeros(T, dtype=torch.int32, device="cuda")
    with pytest.raises(cats.CatsError) as e:
        cats.cats_lm_head_argmax(s["cfg"], dm["final_norm"], dm["w_lm"], resid, T, None, amax, ws[:-1], st)
    assert e.value.status == -4
    nh, hd, Pa = 4, 128, 9000                                       # few heads, long prefix: the merge needs scratch
    q = torch.zeros((T, nh, hd), dtype=torch.bfloat16, device="cuda")
    kv = torch.zeros((Pa + T, nh * hd), dtype=torch.bfloat16, device="cuda")
    out = torch.zeros_like(q)
    with pytest.raises(cats.CatsError) as e:
        cats.cats_tree_attention(q, kv, kv, s["mask"], T, Pa, nh, hd, nh * hd, 0.1, out, None, st)
    assert e.value.status == -4
    with pytest.raises(cats.CatsError) as e:
        cats.cats_tree_attention(q, kv, kv, s["mask"], T, Pa, nh, hd, nh * hd, 0.1, out, ws[:1024], st)
    assert e.value.status == -4
    torch.cuda.synchronize()
    assert int(st.item()) == 0 and torch.equal(resid, before) and torch.all(out == 0)
