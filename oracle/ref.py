"""ctypes binding of the plain-C oracle (``cats_ref.c``).

Test infrastructure only.  bf16 tensors are passed as ``numpy.uint16`` arrays
holding the raw bit patterns; caches are ``float32`` arrays (every bf16 value
is exactly representable), activations handed between steps are ``float64``.
"""
import ctypes as C
import os

import numpy as np

from .build import build as _build

__all__ = [
    "RefCfg", "set_contract", "set_accum32", "to_bf16", "from_bf16", "build_tree_mask", "rmsnorm", "linear",
    "rope_head", "tree_attention", "tree_attention_rows", "verify_layer", "verify_layer_nodes", "embed", "lm_head_argmax", "accept_path",
    "compact_kv", "verify_forward", "n_threads", "typical_stats", "accept_path_typical_def",
    "accept_path_typical",
]

_lib = C.CDLL(_build())


class RefCfg(C.Structure):
    _fields_ = [("hidden", C.c_int32), ("n_heads", C.c_int32), ("head_dim", C.c_int32),
                ("ffn", C.c_int32), ("vocab", C.c_int32), ("n_layers", C.c_int32),
                ("max_seq", C.c_int32), ("rms_eps", C.c_float), ("rope_base", C.c_float)]


class _LayerW(C.Structure):
    _fields_ = [(n, C.c_void_p) for n in
                ("attn_norm", "wq", "wk", "wv", "wo", "mlp_norm", "w_gate", "w_up", "w_down")]


LAYER_FIELDS = tuple(n for n, _ in _LayerW._fields_)


def _p(a):
    return None if a is None else a.ctypes.data_as(C.c_void_p)


def _chk(a, dtype, name):
    a = np.ascontiguousarray(a, dtype=dtype)
    return a


def n_threads() -> int:
    """Number of OpenMP threads the oracle's parallel loops use."""
    env = os.environ.get("OMP_NUM_THREADS")
    if env:
        return int(env)
    return len(os.sched_getaffinity(0))


def set_contract(on: bool) -> None:
    """True: mirror the GPU path's bf16 rounding points.  False: no intermediate rounding."""
    _lib.cats_ref_set_contract(C.c_int(1 if on else 0))


def set_accum32(on: bool) -> None:
    """Sensitivity probe: accumulate the projections in fp32 instead of fp64 (see cats_ref.c)."""
    _lib.cats_ref_set_accum32(C.c_int(1 if on else 0))


_lib.cats_ref_bf16_to_f32.restype = C.c_float
_lib.cats_ref_bf16_to_f32.argtypes = [C.c_uint16]
_lib.cats_ref_f32_to_bf16.restype = C.c_uint16
_lib.cats_ref_f32_to_bf16.argtypes = [C.c_float]


def to_bf16(x) -> np.ndarray:
    """float32 -> bf16 bit patterns, round to nearest even (vectorised restatement of the C helper)."""
    u = np.ascontiguousarray(x, dtype=np.float32).view(np.uint32).astype(np.uint64)
    lsb = (u >> 16) & 1
    r = ((u + 0x7FFF + lsb) >> 16).astype(np.uint16)
    return r


def from_bf16(b) -> np.ndarray:
    return (np.ascontiguousarray(b, dtype=np.uint16).astype(np.uint32) << 16).view(np.float32)


def build_tree_mask(parent, prefix_len):
    parent = _chk(parent, np.int32, "parent")
    T = parent.shape[0]
    mask = np.zeros((T, 2), np.uint64)
    pos = np.zeros(T, np.int32)
    depth = np.zeros(T, np.int32)
    rc = _lib.cats_ref_build_tree_mask(_p(parent), C.c_int32(T), C.c_int32(prefix_len), _p(mask), _p(pos), _p(depth))
    return rc, mask, pos, depth


def rmsnorm(x, g, eps):
    x = _chk(x, np.float32, "x")
    g = _chk(g, np.uint16, "g")
    T, H = x.shape
    out = np.empty((T, H), np.float64)
    _lib.cats_ref_rmsnorm(_p(x), _p(g), C.c_int32(T), C.c_int32(H), C.c_float(eps), _p(out))
    return out


def linear(W, x):
    W = _chk(W, np.uint16, "W")
    x = _chk(x, np.float64, "x")
    n_out, n_in = W.shape
    T = x.shape[0]
    assert x.shape[1] == n_in
    y = np.empty((T, n_out), np.float64)
    _lib.cats_ref_linear(_p(W), C.c_int32(n_out), C.c_int32(n_in), _p(x), C.c_int32(T), _p(y))
    return y


def rope_head(x, pos, base):
    x = np.array(x, dtype=np.float64, copy=True)
    _lib.cats_ref_rope_head(_p(x), C.c_int32(x.shape[0]), C.c_int32(pos), C.c_double(base))
    return x


def tree_attention(q, kc, vc, mask, P, nh, hd, scale, kv_row_stride=None, want_probs=False):
    q = _chk(q, np.float64, "q")
    kc = _chk(kc, np.float32, "kc")
    vc = _chk(vc, np.float32, "vc")
    mask = _chk(mask, np.uint64, "mask")
    T = q.shape[0]
    if kv_row_stride is None:
        kv_row_stride = nh * hd
    assert kc.size >= (P + T) * kv_row_stride and vc.size >= (P + T) * kv_row_stride
    out = np.empty((T, nh, hd), np.float64)
    probs = np.zeros((nh, T, P + T), np.float64) if want_probs else None
    rc = _lib.cats_ref_tree_attention(_p(q), _p(kc), _p(vc), _p(mask), C.c_int32(T), C.c_int32(P),
                                      C.c_int32(nh), C.c_int32(hd), C.c_int64(kv_row_stride),
                                      C.c_double(scale), _p(out), _p(probs))
    assert rc == 0
    return (out, probs) if want_probs else out


def tree_attention_rows(q, kc, vc, mask_rows, T, P, nh, hd, scale):
    """nq query rows, each with its own visibility row over the T tree rows (see cats_ref.c)."""
    q = _chk(q, np.float64, "q")
    kc = _chk(kc, np.float32, "kc")
    vc = _chk(vc, np.float32, "vc")
    mask_rows = _chk(mask_rows, np.uint64, "mask_rows")
    nq = q.shape[0]
    assert mask_rows.shape == (nq, 2) and kc.size >= (P + T) * nh * hd
    out = np.empty((nq, nh, hd), np.float64)
    rc = _lib.cats_ref_tree_attention_rows(_p(q), _p(kc), _p(vc), _p(mask_rows), C.c_int32(nq), C.c_int32(T),
                                           C.c_int32(P), C.c_int32(nh), C.c_int32(hd), C.c_int64(nh * hd),
                                           C.c_double(scale), _p(out), None)
    assert rc == 0, rc
    return out


def _layer_struct(w, keep):
    s = _LayerW()
    for n in LAYER_FIELDS:
        a = _chk(w[n], np.uint16, n)
        keep.append(a)
        setattr(s, n, a.ctypes.data)
    return s


def verify_layer(cfg: RefCfg, w: dict, resid, kc, vc, mask, pos, P, want_q=False):
    """In place on resid (float32 [T,H]) and on kc/vc (float32 [max_seq, nh*hd])."""
    assert resid.dtype == np.float32 and resid.flags.c_contiguous
    assert kc.dtype == np.float32 and kc.flags.c_contiguous and vc.dtype == np.float32 and vc.flags.c_contiguous
    mask = _chk(mask, np.uint64, "mask")
    pos = _chk(pos, np.int32, "pos")
    T = resid.shape[0]
    keep = []
    s = _layer_struct(w, keep)
    q = np.empty((T, cfg.n_heads * cfg.head_dim), np.float64) if want_q else None
    rc = _lib.cats_ref_verify_layer(C.byref(cfg), C.byref(s), _p(resid), _p(kc), _p(vc), _p(mask), _p(pos),
                                    C.c_int32(T), C.c_int32(P), _p(q))
    assert rc == 0, rc
    return q


def verify_layer_nodes(cfg: RefCfg, w: dict, resid, kc, vc, mask, pos, nodes, P):
    """The layer over the tree nodes `nodes` only (ascending).  In place on resid (float32 [m,H]) and on the cache rows
    P + nodes[j]; mask [T,2] and pos [T] describe the whole tree."""
    assert resid.dtype == np.float32 and resid.flags.c_contiguous
    assert kc.dtype == np.float32 and kc.flags.c_contiguous and vc.dtype == np.float32 and vc.flags.c_contiguous
    mask = _chk(mask, np.uint64, "mask")
    pos = _chk(pos, np.int32, "pos")
    nodes = _chk(nodes, np.int32, "nodes")
    assert resid.shape[0] == nodes.shape[0]
    keep = []
    s = _layer_struct(w, keep)
    rc = _lib.cats_ref_verify_layer_nodes(C.byref(cfg), C.byref(s), _p(resid), _p(kc), _p(vc), _p(mask), _p(pos),
                                          _p(nodes), C.c_int32(nodes.shape[0]), C.c_int32(pos.shape[0]), C.c_int32(P))
    return rc


def embed(E, tokens):
    E = _chk(E, np.uint16, "E")
    tokens = _chk(tokens, np.int32, "tokens")
    out = np.empty((tokens.shape[0], E.shape[1]), np.float32)
    _lib.cats_ref_embed(_p(E), _p(tokens), C.c_int32(tokens.shape[0]), C.c_int32(E.shape[1]), _p(out))
    return out


def lm_head_argmax(cfg: RefCfg, final_norm, w_lm, resid, want_logits=True):
    final_norm = _chk(final_norm, np.uint16, "final_norm")
    w_lm = _chk(w_lm, np.uint16, "w_lm")
    resid = _chk(resid, np.float32, "resid")
    T = resid.shape[0]
    logits = np.empty((T, cfg.vocab), np.float32) if want_logits else None
    amax = np.empty(T, np.int32)
    margin = np.empty(T, np.float32)
    rc = _lib.cats_ref_lm_head_argmax(C.byref(cfg), _p(final_norm), _p(w_lm), _p(resid), C.c_int32(T),
                                      _p(logits), _p(amax), _p(margin))
    assert rc == 0
    return logits, amax, margin


def accept_path(parent, tokens, argmax):
    parent = _chk(parent, np.int32, "parent")
    tokens = _chk(tokens, np.int32, "tokens")
    argmax = _chk(argmax, np.int32, "argmax")
    T = parent.shape[0]
    path = np.full(T, -1, np.int32)
    out = np.full(T, -1, np.int32)
    pl = C.c_int32(0)
    no = C.c_int32(0)
    rc = _lib.cats_ref_accept_path(_p(parent), _p(tokens), _p(argmax), C.c_int32(T), _p(path), C.byref(pl),
                                   _p(out), C.byref(no))
    assert rc == 0
    return path[:pl.value].copy(), out[:no.value].copy()


def typical_stats(logits, temperature, parent, tokens):
    """Per-node softmax statistics at the given temperature: (lse f32 [T], entropy f32 [T], cand_logit f32 [T],
    prob f64 [T] = p_parent(token))."""
    logits = _chk(logits, np.float32, "logits")
    parent = _chk(parent, np.int32, "parent")
    tokens = _chk(tokens, np.int32, "tokens")
    T, V = logits.shape
    lse = np.empty(T, np.float32)
    ent = np.empty(T, np.float32)
    cand = np.empty(T, np.float32)
    prob = np.empty(T, np.float64)
    rc = _lib.cats_ref_typical_stats(_p(logits), C.c_int32(T), C.c_int32(V), C.c_double(temperature), _p(parent),
                                     _p(tokens), _p(lse), _p(ent), _p(cand), _p(prob))
    assert rc == 0, rc
    return lse, ent, cand, prob


def _walk_out(T):
    return np.full(T, -1, np.int32), np.full(T, -1, np.int32), C.c_int32(0), C.c_int32(0)


def accept_path_typical_def(parent, tokens, argmax, logits, temperature, eps, delta):
    """Typical acceptance from its definition (fp64, on the logits).  Returns (path, out_tokens)."""
    parent = _chk(parent, np.int32, "parent")
    tokens = _chk(tokens, np.int32, "tokens")
    argmax = _chk(argmax, np.int32, "argmax")
    logits = _chk(logits, np.float32, "logits")
    T, V = logits.shape
    path, out, pl, no = _walk_out(T)
    rc = _lib.cats_ref_accept_path_typical_def(_p(parent), _p(tokens), _p(argmax), _p(logits), C.c_int32(T), C.c_int32(V),
                                               C.c_double(temperature), C.c_double(eps), C.c_double(delta), _p(path),
                                               C.byref(pl), _p(out), C.byref(no))
    assert rc == 0, rc
    return path[:pl.value].copy(), out[:no.value].copy()


def accept_path_typical(parent, tokens, argmax, cand_logit, lse, entropy, inv_temperature, log_eps, log_delta):
    """The same walk from fp32 statistics, verdict in the log domain in fp32 (see cats_ref.c)."""
    parent = _chk(parent, np.int32, "parent")
    tokens = _chk(tokens, np.int32, "tokens")
    argmax = _chk(argmax, np.int32, "argmax")
    cand_logit = _chk(cand_logit, np.float32, "cand")
    lse = _chk(lse, np.float32, "lse")
    entropy = _chk(entropy, np.float32, "entropy")
    T = parent.shape[0]
    path, out, pl, no = _walk_out(T)
    rc = _lib.cats_ref_accept_path_typical(_p(parent), _p(tokens), _p(argmax), _p(cand_logit), _p(lse), _p(entropy),
                                           C.c_int32(T), C.c_float(inv_temperature), C.c_float(log_eps),
                                           C.c_float(log_delta), _p(path), C.byref(pl), _p(out), C.byref(no))
    assert rc == 0, rc
    return path[:pl.value].copy(), out[:no.value].copy()


def compact_kv(kc, vc, P, path):
    """kc, vc: arrays [n_layers, rows, row_elems] of any dtype, compacted in place."""
    assert kc.flags.c_contiguous and vc.flags.c_contiguous and kc.dtype == vc.dtype and kc.ndim == 3
    path = _chk(path, np.int32, "path")
    L, S, R = kc.shape
    n = path.shape[0]
    src = np.empty(n, np.int32)
    dst = np.empty(n, np.int32)
    new_len = C.c_int32(0)
    rc = _lib.cats_ref_compact_kv(_p(kc), _p(vc), C.c_int32(L), C.c_int64(S * R), C.c_int64(R),
                                  C.c_int32(kc.dtype.itemsize), C.c_int32(P), _p(path), C.c_int32(n),
                                  C.byref(new_len), _p(src), _p(dst))
    return rc, new_len.value, src, dst


def verify_forward(cfg: RefCfg, layers, embed_w, final_norm, w_lm, parent, tokens, P, kc, vc,
                   hidden_in=None, want_logits=True):
    """Whole Stage-3 forward.  kc, vc float32 [n_layers, max_seq, nh*hd], updated in place.

    Returns (logits or None, argmax, margin, resid)."""
    parent = _chk(parent, np.int32, "parent")
    tokens = _chk(tokens, np.int32, "tokens")
    T = parent.shape[0]
    assert kc.dtype == np.float32 and kc.flags.c_contiguous and vc.dtype == np.float32 and vc.flags.c_contiguous
    assert kc.shape == (cfg.n_layers, cfg.max_seq, cfg.n_heads * cfg.head_dim)
    keep = []
    arr = (_LayerW * cfg.n_layers)()
    for l in range(cfg.n_layers):
        arr[l] = _layer_struct(layers[l], keep)
    embed_w = None if embed_w is None else _chk(embed_w, np.uint16, "embed")
    final_norm = _chk(final_norm, np.uint16, "final_norm")
    w_lm = _chk(w_lm, np.uint16, "w_lm")
    hidden_in = None if hidden_in is None else _chk(hidden_in, np.float32, "hidden_in")
    logits = np.empty((T, cfg.vocab), np.float32) if want_logits else None
    amax = np.empty(T, np.int32)
    margin = np.empty(T, np.float32)
    resid = np.empty((T, cfg.hidden), np.float32)
    rc = _lib.cats_ref_verify_forward(C.byref(cfg), arr, _p(embed_w), _p(final_norm), _p(w_lm), _p(parent),
                                      _p(tokens), _p(hidden_in), C.c_int32(T), C.c_int32(P), _p(kc), _p(vc),
                                      _p(logits), _p(amax), _p(margin), _p(resid))
    assert rc == 0, rc
    return logits, amax, margin, resid
