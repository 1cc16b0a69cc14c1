"""The draft-stage shape of a cycle (Algorithm 1, Stage 1: gamma sequential one-token passes through layers 1..L_DM): the
same kernels at T = 1 over a layer range, with the prefix growing by one row per pass.  The draft adapter that turns the
hidden state into the next draft token needs trained weights and is outside this build, so the draft tokens are given.

Checked against the oracle's own sequential passes, and against ONE chain-tree pass over the same tokens (tree
verification of a chain is sequential decoding): the cache rows the two leave behind agree."""
import numpy as np
import pytest
import torch

import oracle
from paper_2605_11186_b200 import inputs as gen
from helpers import ref_cfg, np_model, cache_to_f32
from test_gpu_parity import TOL, dev, dev_model, bf16_ulp_close, contract_floor

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def cats():
    from paper_2605_11186_b200 import binding
    assert torch.cuda.is_available()
    return binding


def _case(cats, m_full, L_DM, gamma, P, tag):
    m = m_full.replace(n_layers=L_DM)
    model = gen.make_model(m, tag)
    nm = np_model(model)
    max_seq = P + gamma + 8
    kc, vc = gen.make_kv_prefix(m, L_DM, max_seq, P, tag)
    tokens = gen.uniform_tokens(gamma, m.vocab, tag, "draft")
    rcfg = ref_cfg(m, max_seq)
    one = np.array([-1], np.int32)

    # oracle: gamma one-token passes (twice: fp64- and fp32-accumulated projections bound what rounding alone can do)
    def run():
        r_k, r_v = cache_to_f32(kc), cache_to_f32(vc)
        hid, lg = [], []
        for s in range(gamma):
            logits, amax, margin, resid = oracle.verify_forward(rcfg, nm["layers"], nm["embed"], nm["final_norm"], nm["w_lm"],
                                                                one, tokens[s:s + 1], P + s, r_k, r_v)
            hid.append(resid[0].copy())
            lg.append(logits[0].copy())
        return np.stack(hid), np.stack(lg), r_k, r_v
    (r_hidden, r_logits, r_k, r_v), floor = contract_floor(run)
    tol_h, tol_l = max(TOL, 3.0 * floor[0]), max(TOL, 3.0 * floor[1])

    # GPU: the same passes, one forward object whose prefix length advances
    dm = cats.pack_model(dev_model(model))
    d_k, d_v = kc.cuda(), vc.cuda()
    fwd = cats.VerifyForward(m, dm, d_k, d_v, 1, P, want_logits=True, compact=False)
    d_one = dev(one)
    for s in range(gamma):
        fwd.set_prefix_len(P + s)
        fwd.run(d_one, dev(tokens[s:s + 1]))
        torch.cuda.synchronize()
        assert int(fwd.status.item()) == 0
        assert np.abs(fwd.resid.cpu().numpy()[0] - r_hidden[s]).max() <= tol_h, (s, tol_h)
        assert np.abs(fwd.logits.cpu().numpy()[0] - r_logits[s]).max() <= tol_l, (s, tol_l)
        assert int(fwd.pos[0]) == P + s
    # layer 0 sees identical inputs on both sides: its rows agree to one bf16 ulp; deeper layers inherit the rounding
    # spread of the layers before them
    tol_kv = max(TOL, 3.0 * max(floor[2], floor[3]))
    for l in range(L_DM):
        for got, want in ((d_k[l], r_k[l]), (d_v[l], r_v[l])):
            if l == 0:
                nbad, maxerr = bf16_ulp_close(got[P:P + gamma], want[P:P + gamma])
                assert nbad == 0, (l, nbad, maxerr)
            assert np.abs(got[P:P + gamma].float().cpu().numpy() - want[P:P + gamma]).max() <= tol_kv + 2.0 ** -5
            assert torch.all(got[P + gamma:] == 0)

    # one chain-tree pass over the same tokens leaves (within rounding) the same rows
    c_k, c_v = kc.cuda(), vc.cuda()
    chain = cats.VerifyForward(m, dm, c_k, c_v, gamma, P, want_logits=False, compact=False)
    chain.run(dev(gen.tree_chain(gamma)), dev(tokens))
    torch.cuda.synchronize()
    assert int(chain.status.item()) == 0
    nbad, maxerr = bf16_ulp_close(c_k[0, P:P + gamma], r_k[0, P:P + gamma])
    assert nbad == 0, (nbad, maxerr)
    for l in range(L_DM):
        assert np.abs(c_k[l, P:P + gamma].float().cpu().numpy() - r_k[l, P:P + gamma]).max() <= tol_kv + 2.0 ** -5
    assert np.abs(chain.resid.cpu().numpy() - r_hidden).max() <= tol_h


def test_draft_passes_tiny(cats):
    _case(cats, gen.TINY, 2, 5, 77, "draft_tiny")


def test_draft_passes_7b_shape(cats):
    """Three draft layers of the 7B shape (the paper's B_draft = 3 layers), gamma = 3, prefix 512."""
    _case(cats, gen.LLAMA_7B, 3, 3, 512, "draft_7b")
