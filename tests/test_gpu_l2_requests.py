"""The requests into L2 that the attention and norm kernels issue for the projections after them (see
cats_debug_l2_warm in include/cats_debug.h) only move bytes earlier: logits, accepted path and compacted cache must be
the same bit for bit whether they are issued as built in, not at all, or for every matrix at once."""
import numpy as np
import pytest
import torch

from paper_2605_11186_b200 import inputs as gen

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def cats():
    from paper_2605_11186_b200 import binding
    assert torch.cuda.is_available()
    return binding


def _run(cats, shape, model, T, P, tag):
    kc, vc = gen.make_kv_prefix(shape, shape.n_layers, P + T + 8, P, tag, device="cuda")
    parent, _ = gen.tree_topk_shape(T, gen.topk_k_for(T))
    tokens = gen.uniform_tokens(T, shape.vocab, tag, T)
    fwd = cats.VerifyForward(shape, model, kc, vc, T, P, want_logits=True, compact=True)
    fwd.run(torch.from_numpy(parent).cuda(), torch.from_numpy(tokens).cuda())
    torch.cuda.synchronize()
    assert int(fwd.status.item()) == 0
    return (fwd.logits.cpu().numpy().copy(), fwd.path.cpu().numpy().copy(), fwd.scalars.cpu().numpy().copy(),
            kc.cpu().view(torch.int16).numpy().copy(), vc.cpu().view(torch.int16).numpy().copy())


@pytest.mark.parametrize("T", [1, 16, 64, 100])
def test_l2_requests_change_no_result(cats, T):
    # wide enough that every matrix has several 32 KB units, small enough to run in a second
    shape = gen.ModelShape(hidden=1024, n_heads=8, head_dim=128, ffn=2816, vocab=4096, n_layers=3)
    model = cats.pack_model(gen.make_model(shape, "l2req", device="cuda"), free_source=True)
    P = 300
    try:
        ref = _run(cats, shape, model, T, P, "l2req")
        for which in range(5):
            cats.l2_warm(which, 0)
        off = _run(cats, shape, model, T, P, "l2req")
        for which in range(5):
            cats.l2_warm(which, 2, which % 2)
        every = _run(cats, shape, model, T, P, "l2req")
    finally:
        for which, period in enumerate((0, -1, 0, -1, 0)):
            cats.l2_warm(which, period)
    for name, a, b, c in zip(("logits", "path", "scalars", "kcache", "vcache"), ref, off, every):
        assert np.array_equal(a, b), name + ": differs with the requests switched off"
        assert np.array_equal(a, c), name + ": differs with requests for every matrix"
