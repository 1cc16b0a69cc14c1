"""Thin ctypes binding of ``libcats.so``: argument marshalling only.

Every function takes torch CUDA tensors (used purely as device memory), passes their data pointers and the
current CUDA stream to the C-ABI entry point of the same name, and raises ``CatsError`` on a negative
status.  There is no fallback: if the library cannot be loaded, importing this module fails.
"""
import ctypes as C
import os

import torch

from . import build as _build

_HERE = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(_HERE, "libcats.so")
# CATS_LIBRARY: another build of the same library (timeline.py sets it to the measurement build before importing this)
if os.environ.get("CATS_LIBRARY"):
    LIB_PATH = os.environ["CATS_LIBRARY"]
    if not os.path.exists(LIB_PATH):
        raise FileNotFoundError("CATS_LIBRARY=%s does not exist" % LIB_PATH)
elif not os.path.exists(LIB_PATH):
    _build.build()
lib = C.CDLL(LIB_PATH)

MAX_TREE = 128


class CatsError(RuntimeError):
    def __init__(self, status, where):
        self.status = status
        super().__init__("%s: %s (%d)" % (where, lib.cats_status_string(status).decode(), status))


class ModelCfg(C.Structure):
    _fields_ = [("hidden", C.c_int32), ("n_heads", C.c_int32), ("head_dim", C.c_int32), ("ffn", C.c_int32),
                ("vocab", C.c_int32), ("n_layers", C.c_int32), ("max_seq", C.c_int32), ("rms_eps", C.c_float),
                ("rope_base", C.c_float)]


LAYER_FIELDS = ("attn_norm", "wqkv", "wo", "mlp_norm", "w_gate_up", "w_down")


class LayerWeights(C.Structure):
    _fields_ = [(n, C.c_void_p) for n in LAYER_FIELDS]


class ForwardArgs(C.Structure):
    _fields_ = [("cfg", C.POINTER(ModelCfg)), ("layers", C.POINTER(LayerWeights)), ("d_embed", C.c_void_p),
                ("d_final_norm", C.c_void_p), ("d_w_lm", C.c_void_p), ("d_kcache", C.c_void_p), ("d_vcache", C.c_void_p),
                ("d_hidden_in", C.c_void_p), ("T", C.c_int32), ("prefix_len", C.c_int32), ("compact", C.c_int32),
                ("d_mask", C.c_void_p), ("d_pos", C.c_void_p), ("d_depth", C.c_void_p), ("d_resid", C.c_void_p),
                ("d_logits", C.c_void_p), ("d_argmax", C.c_void_p), ("d_path", C.c_void_p), ("d_out_tokens", C.c_void_p),
                ("d_scalars", C.c_void_p), ("d_ws", C.c_void_p), ("ws_bytes", C.c_size_t), ("d_status", C.c_void_p),
                ("accept_mode", C.c_int32), ("inv_temperature", C.c_float), ("log_eps", C.c_float), ("log_delta", C.c_float),
                ("d_typical", C.c_void_p)]


ACCEPT_GREEDY, ACCEPT_TYPICAL = 0, 1


lib.cats_status_string.restype = C.c_char_p
lib.cats_status_string.argtypes = [C.c_int]
lib.cats_version.restype = C.c_int
lib.cats_last_launch_count.restype = C.c_int
lib.cats_workspace_bytes.restype = C.c_size_t
lib.cats_workspace_bytes.argtypes = [C.POINTER(ModelCfg), C.c_int32, C.c_int32]
_vp, _i32, _i64 = C.c_void_p, C.c_int32, C.c_int64
lib.cats_build_tree_mask.argtypes = [_vp, _i32, _i32, _vp, _vp, _vp, _vp, _vp]
lib.cats_embed_tokens.argtypes = [_vp, _vp, _i32, _i32, _i32, _vp, _vp, _vp]
lib.cats_verify_layer.argtypes = [C.POINTER(ModelCfg), C.POINTER(LayerWeights), _vp, _vp, _vp, _vp, _vp, _i32, _i32, _vp,
                                  C.c_size_t, _vp, _vp]
lib.cats_verify_layer_nodes.argtypes = [C.POINTER(ModelCfg), C.POINTER(LayerWeights), _vp, _vp, _vp, _vp, _vp, _vp, _i32, _i32,
                                        _i32, _vp, C.c_size_t, _vp, _vp]
lib.cats_tree_attention.argtypes = [_vp, _vp, _vp, _vp, _i32, _i32, _i32, _i32, _i64, C.c_float, _vp, _vp, C.c_size_t, _vp, _vp]
lib.cats_lm_head_argmax.argtypes = [C.POINTER(ModelCfg), _vp, _vp, _vp, _i32, _vp, _vp, _vp, C.c_size_t, _vp, _vp]
lib.cats_accept_path.argtypes = [_vp, _vp, _vp, _i32, _vp, _vp, _vp, _vp, _vp, _vp]
lib.cats_lm_head_typical.argtypes = [C.POINTER(ModelCfg), _vp, _vp, _vp, _vp, _vp, _i32, C.c_float, _vp, _vp, _vp, _vp, _vp, _vp,
                                     C.c_size_t, _vp, _vp]
lib.cats_accept_path_typical.argtypes = [_vp, _vp, _vp, _vp, _vp, _vp, _i32, C.c_float, C.c_float, C.c_float, _vp, _vp, _vp,
                                         _vp, _vp, _vp]
lib.cats_compact_kv.argtypes = [_vp, _vp, _i32, _i64, _i64, _i32, _vp, _vp, _vp, _vp, _vp, _vp, _vp]
lib.cats_verify_forward.argtypes = [C.POINTER(ForwardArgs), _vp, _vp, _vp]
lib.cats_verify_forward_host.argtypes = [C.POINTER(ForwardArgs), _vp, _vp, _vp, _vp, _vp, _vp, _vp, _vp]
lib.cats_tp_attention_half.argtypes = [C.POINTER(ModelCfg), C.POINTER(LayerWeights), _vp, _vp, _vp, _vp, _vp, _vp, _i32, _i32, _vp,
                                       _vp, C.c_size_t, _vp, _vp]
lib.cats_tp_mlp_half.argtypes = [C.POINTER(ModelCfg), C.POINTER(LayerWeights), _vp, _vp, _i32, _vp, _vp, C.c_size_t, _vp, _vp]
lib.cats_tp_lm_head_shard.argtypes = [C.POINTER(ModelCfg), _vp, _vp, _vp, _vp, _i32, _i32, _vp, _vp, _vp, _vp, C.c_size_t, _vp, _vp]
lib.cats_tp_argmax_merge.argtypes = [_vp, _vp, _i32, _i32, _vp, _vp]
lib.cats_packed_weight_bytes.restype = C.c_size_t
lib.cats_packed_weight_bytes.argtypes = [_i32, _i32, _i32, _i32]
lib.cats_pack_weights.argtypes = [C.POINTER(C.c_void_p), _i32, _i32, _i32, _i32, _vp, _vp]


def _ptr(t):
    if t is None:
        return None
    if isinstance(t, torch.Tensor):
        assert t.is_contiguous(), "tensors handed to libcats must be contiguous"
        return t.data_ptr()
    return int(t)


def _stream():
    return torch.cuda.current_stream().cuda_stream


def _check(rc, where):
    if rc != 0:
        raise CatsError(rc, where)


def model_cfg(shape, max_seq, n_layers=None) -> ModelCfg:
    """``shape``: any object with hidden, n_heads, head_dim, ffn, vocab, n_layers, rms_eps, rope_base."""
    return ModelCfg(shape.hidden, shape.n_heads, shape.head_dim, shape.ffn, shape.vocab,
                    shape.n_layers if n_layers is None else n_layers, max_seq, shape.rms_eps, shape.rope_base)


def pack_weights(mats, layout: int) -> torch.Tensor:
    """cats_pack_weights: ``mats`` is a list of 1-3 bf16 CUDA matrices of identical shape [rows][cols]
    (nn.Linear layout).  Returns the packed buffer (uint8 CUDA tensor, 1024-byte aligned)."""
    rows, cols = mats[0].shape
    for m in mats:
        assert m.is_cuda and m.dtype == torch.bfloat16 and m.is_contiguous() and tuple(m.shape) == (rows, cols)
    n = int(lib.cats_packed_weight_bytes(len(mats), layout, rows, cols))
    if n == 0:
        raise CatsError(-1, "cats_packed_weight_bytes")
    buf = torch.empty(n + 1024, dtype=torch.uint8, device=mats[0].device)
    off = (-buf.data_ptr()) % 1024
    out = buf[off:off + n]
    ptrs = (C.c_void_p * len(mats))(*[m.data_ptr() for m in mats])
    _check(lib.cats_pack_weights(ptrs, len(mats), layout, rows, cols, out.data_ptr(), _stream()), "cats_pack_weights")
    return out


def pack_layer(w: dict) -> dict:
    """nn.Linear-layout layer weights (wq, wk, wv, wo, w_gate, w_up, w_down, attn_norm, mlp_norm) -> packed layer."""
    return {"attn_norm": w["attn_norm"].contiguous(), "mlp_norm": w["mlp_norm"].contiguous(),
            "wqkv": pack_weights([w["wq"], w["wk"], w["wv"]], 0), "wo": pack_weights([w["wo"]], 0),
            "w_gate_up": pack_weights([w["w_gate"], w["w_up"]], 1), "w_down": pack_weights([w["w_down"]], 0)}


def pack_model(model: dict, free_source: bool = False) -> dict:
    """Packs every projection of a model dict (layers, w_lm); embed and final_norm are kept as they are."""
    out = {"layers": []}
    for w in model["layers"]:
        out["layers"].append(pack_layer(w))
        if free_source:
            for k in ("wq", "wk", "wv", "wo", "w_gate", "w_up", "w_down"):
                w.pop(k, None)
    for k in ("embed", "final_norm", "shape"):
        if k in model:
            out[k] = model[k]
    if "w_lm" in model:
        out["w_lm"] = pack_weights([model["w_lm"]], 0)
        if free_source:
            model.pop("w_lm")
    torch.cuda.synchronize()
    return out


def layer_weights(w: dict) -> LayerWeights:
    """``w``: a packed layer (see pack_layer)."""
    s = LayerWeights()
    for n in LAYER_FIELDS:
        t = w[n]
        assert t.is_cuda and t.is_contiguous(), n
        setattr(s, n, t.data_ptr())
    return s


def new_status(device="cuda") -> torch.Tensor:
    return torch.zeros(1, dtype=torch.int32, device=device)


def workspace_bytes(cfg: ModelCfg, T: int, max_prefix: int) -> int:
    return int(lib.cats_workspace_bytes(C.byref(cfg), T, max_prefix))


def new_workspace(cfg: ModelCfg, T: int, max_prefix: int, device="cuda") -> torch.Tensor:
    n = workspace_bytes(cfg, T, max_prefix)
    if n == 0:
        raise CatsError(-3, "cats_workspace_bytes")
    buf = torch.empty(n + 1024, dtype=torch.uint8, device=device)
    off = (-buf.data_ptr()) % 1024
    return buf[off:off + n]


def stage_mask(mask: int) -> None:
    """Measurement / bring-up hook: bit i enables stage i of every decoder layer (0 norm1, 1 qkv, 2 attention,
    3 o-proj, 4 norm2, 5 gate/up, 6 down).  0x7f is normal operation."""
    lib.cats_debug_stage_mask(C.c_uint(mask))


def attention_kernel(which: int) -> None:
    """cats_debug_attention_kernel: -1 by shape (default), 0 the mma.sync kernel, 1 the tcgen05 kernel, 2 the tcgen05
    kernel with two softmax threads per query row instead of four."""
    lib.cats_debug_attention_kernel(C.c_int(which))


def wait_limit_ns(ns: int) -> None:
    """cats_debug_wait_limit_ns: limit of the bounded device-side waits on the current device (0: the default, 1 s)."""
    _check(lib.cats_debug_wait_limit_ns(C.c_ulonglong(ns)), "cats_debug_wait_limit_ns")


def inject_fault(which: int) -> None:
    """cats_debug_inject_fault: 0 none, 1 a projection's contributors keep their ready flags, 2 the attention loader
    never copies Q."""
    lib.cats_debug_inject_fault(C.c_int(which))


def l2_warm(which: int, period: int, phase: int = 0) -> None:
    """cats_debug_l2_warm: which weights the kernels that leave HBM idle request into L2 (0 attention -> O, 1 attention ->
    gate/up, 2 attention -> down, 3 norm before QKV -> QKV, 4 norm before gate/up -> gate/up); every period-th 32 KB unit
    from unit ``phase``; period 0 none, -1 the built-in choice."""
    lib.cats_debug_l2_warm(C.c_int(which), C.c_int(period), C.c_int(phase))


TIMELINE_SLOTS = {0: 512, 1: 128, 2: 256}     # launch slots per kernel (projection, tcgen05 attention, register norm)


def timeline(kernel: int):
    """cats_debug_timeline: the stamps of the given kernel as an int64 array [slots][160][16] (ns, zero = not written).
    Only the measurement build records them (CatsError UNSUPPORTED otherwise)."""
    import numpy as np
    a = np.zeros((TIMELINE_SLOTS[kernel], 160, 16), dtype=np.uint64)
    _check(lib.cats_debug_timeline(C.c_int(kernel), C.c_void_p(a.ctypes.data), C.c_size_t(a.nbytes)), "cats_debug_timeline")
    return a.astype(np.int64)


def timeline_clear() -> None:
    for k in TIMELINE_SLOTS:
        _check(lib.cats_debug_timeline(C.c_int(k), None, C.c_size_t(0)), "cats_debug_timeline")


def workspace_layout(cfg: ModelCfg, T: int) -> dict:
    """Byte offsets of the intermediate buffers inside the workspace (for tests that inspect them)."""
    out = (C.c_size_t * 8)()
    _check(lib.cats_debug_workspace_layout(C.byref(cfg), T, out), "cats_debug_workspace_layout")
    return dict(xn=out[0], q=out[1], o=out[2], act=out[3], part=out[4], part_stride=out[5], pieces_o=out[6],
                pieces_down=out[7])


def unpack_activation(buf: torch.Tensor, T: int, K: int) -> torch.Tensor:
    """Reads a packed activation buffer (uint8 view of the workspace) back as a [T][K] bf16 tensor (tests only)."""
    n_pad = (T + 15) // 16 * 16
    n_kb = (K + 63) // 64
    x = buf[:n_kb * n_pad * 128].view(torch.bfloat16).view(n_kb, n_pad // 8, 8, 8, 8)   # kb, row group, row, chunk, elem
    r = torch.arange(8, device=buf.device)
    c = torch.arange(8, device=buf.device)
    phys = (c[None, :] ^ r[:, None])                                                  # [row][logical chunk] -> physical
    x = torch.gather(x, 3, phys[None, None, :, :, None].expand(n_kb, n_pad // 8, 8, 8, 8))
    x = x.permute(1, 2, 0, 3, 4).reshape(n_pad, n_kb * 64)
    return x[:T, :K].contiguous()


def last_launch_count() -> int:
    return int(lib.cats_last_launch_count())


def cats_build_tree_mask(parent, prefix_len, mask, pos, depth, status):
    _check(lib.cats_build_tree_mask(_ptr(parent), parent.numel(), prefix_len, _ptr(mask), _ptr(pos), _ptr(depth),
                                    _ptr(status), _stream()), "cats_build_tree_mask")


def cats_embed_tokens(embed, tokens, resid, status):
    _check(lib.cats_embed_tokens(_ptr(embed), _ptr(tokens), tokens.numel(), embed.shape[1], embed.shape[0], _ptr(resid),
                                 _ptr(status), _stream()), "cats_embed_tokens")


def cats_verify_layer(cfg, w: LayerWeights, resid, kcache, vcache, mask, pos, T, prefix_len, ws, status):
    _check(lib.cats_verify_layer(C.byref(cfg), C.byref(w), _ptr(resid), _ptr(kcache), _ptr(vcache), _ptr(mask), _ptr(pos), T,
                                 prefix_len, _ptr(ws), ws.numel(), _ptr(status), _stream()), "cats_verify_layer")


def cats_verify_layer_nodes(cfg, w: LayerWeights, resid, kcache, vcache, mask, pos, nodes, T, prefix_len, ws, status):
    """The layer over the tree nodes `nodes` (int32 device tensor, ascending) of a tree of T nodes; resid [len(nodes), H]."""
    _check(lib.cats_verify_layer_nodes(C.byref(cfg), C.byref(w), _ptr(resid), _ptr(kcache), _ptr(vcache), _ptr(mask), _ptr(pos),
                                       _ptr(nodes), nodes.numel(), T, prefix_len, _ptr(ws), ws.numel(), _ptr(status), _stream()),
           "cats_verify_layer_nodes")


def cats_tree_attention(q, k, v, mask, T, prefix_len, n_heads, head_dim, kv_row_stride, scale, out, ws, status):
    _check(lib.cats_tree_attention(_ptr(q), _ptr(k), _ptr(v), _ptr(mask), T, prefix_len, n_heads, head_dim, kv_row_stride,
                                   scale, _ptr(out), _ptr(ws), 0 if ws is None else ws.numel(), _ptr(status), _stream()),
           "cats_tree_attention")


STATIC_SCRATCH_BYTES = 1 << 20
lib.cats_tree_attention_static.argtypes = [_vp, _vp, _vp, _vp, _i32, _i32, _i32, _i32, _i64, C.c_float, _vp, _vp, _vp]


def cats_tree_attention_static(q, k, v, mask, T, prefix_len, n_heads, head_dim, kv_row_stride, scale, out, status):
    """cats_tree_attention without a workspace: the scratch is the fixed array inside the library (for callers that
    cannot allocate).  Raises CatsError(-4) if the problem needs more than STATIC_SCRATCH_BYTES of partial results."""
    _check(lib.cats_tree_attention_static(_ptr(q), _ptr(k), _ptr(v), _ptr(mask), T, prefix_len, n_heads, head_dim,
                                          kv_row_stride, scale, _ptr(out), _ptr(status), _stream()),
           "cats_tree_attention_static")


def cats_lm_head_argmax(cfg, final_norm, w_lm, resid, T, logits, argmax, ws, status):
    _check(lib.cats_lm_head_argmax(C.byref(cfg), _ptr(final_norm), _ptr(w_lm), _ptr(resid), T, _ptr(logits), _ptr(argmax),
                                   _ptr(ws), ws.numel(), _ptr(status), _stream()), "cats_lm_head_argmax")


def cats_lm_head_typical(cfg, final_norm, w_lm, resid, parent, tokens, T, inv_temperature, logits, argmax, lse, entropy,
                         cand_logit, ws, status):
    _check(lib.cats_lm_head_typical(C.byref(cfg), _ptr(final_norm), _ptr(w_lm), _ptr(resid), _ptr(parent), _ptr(tokens), T,
                                    float(inv_temperature), _ptr(logits), _ptr(argmax), _ptr(lse), _ptr(entropy),
                                    _ptr(cand_logit), _ptr(ws), ws.numel(), _ptr(status), _stream()), "cats_lm_head_typical")


def cats_accept_path_typical(parent, tokens, argmax, cand_logit, lse, entropy, T, inv_temperature, log_eps, log_delta, path,
                             path_len, out_tokens, n_out, status):
    _check(lib.cats_accept_path_typical(_ptr(parent), _ptr(tokens), _ptr(argmax), _ptr(cand_logit), _ptr(lse), _ptr(entropy),
                                        T, float(inv_temperature), float(log_eps), float(log_delta), _ptr(path),
                                        _ptr(path_len), _ptr(out_tokens), _ptr(n_out), _ptr(status), _stream()),
           "cats_accept_path_typical")


def cats_accept_path(parent, tokens, argmax, T, path, path_len, out_tokens, n_out, status):
    _check(lib.cats_accept_path(_ptr(parent), _ptr(tokens), _ptr(argmax), T, _ptr(path), _ptr(path_len), _ptr(out_tokens),
                                _ptr(n_out), _ptr(status), _stream()), "cats_accept_path")


def cats_compact_kv(kcache, vcache, n_layers, layer_stride, row_elems, prefix_len, path, path_len, new_len, src_rows,
                    dst_rows, status):
    _check(lib.cats_compact_kv(_ptr(kcache), _ptr(vcache), n_layers, layer_stride, row_elems, prefix_len, _ptr(path),
                               _ptr(path_len), _ptr(new_len), _ptr(src_rows), _ptr(dst_rows), _ptr(status), _stream()),
           "cats_compact_kv")


def cats_tp_attention_half(cfg, w: LayerWeights, resid, pending, kcache, vcache, mask, pos, T, prefix_len, partial_out, ws, status):
    _check(lib.cats_tp_attention_half(C.byref(cfg), C.byref(w), _ptr(resid), _ptr(pending), _ptr(kcache), _ptr(vcache), _ptr(mask),
                                      _ptr(pos), T, prefix_len, _ptr(partial_out), _ptr(ws), ws.numel(), _ptr(status), _stream()),
           "cats_tp_attention_half")


def cats_tp_mlp_half(cfg, w: LayerWeights, resid, pending, T, partial_out, ws, status):
    _check(lib.cats_tp_mlp_half(C.byref(cfg), C.byref(w), _ptr(resid), _ptr(pending), T, _ptr(partial_out), _ptr(ws), ws.numel(),
                                _ptr(status), _stream()), "cats_tp_mlp_half")


def cats_tp_lm_head_shard(cfg, final_norm, w_lm, resid, pending, T, vocab_offset, logits, max_out, argmax_out, ws, status):
    _check(lib.cats_tp_lm_head_shard(C.byref(cfg), _ptr(final_norm), _ptr(w_lm), _ptr(resid), _ptr(pending), T, vocab_offset,
                                     _ptr(logits), _ptr(max_out), _ptr(argmax_out), _ptr(ws), ws.numel(), _ptr(status), _stream()),
           "cats_tp_lm_head_shard")


def cats_tp_argmax_merge(max_all, idx_all, n_shards, T, argmax):
    _check(lib.cats_tp_argmax_merge(_ptr(max_all), _ptr(idx_all), n_shards, T, _ptr(argmax), _stream()), "cats_tp_argmax_merge")


class VerifyForward:
    """Holds the argument block of ``cats_verify_forward`` for one model / tree size: device buffers for
    every output plus the workspace, all allocated once here (the library itself allocates nothing)."""

    def __init__(self, shape, model: dict, kcache, vcache, T: int, prefix_len: int, want_logits=True, compact=True,
                 hidden_in=None, typical=None):
        """typical: None for greedy acceptance, else (inv_temperature, log_eps, log_delta) as float32 values."""
        dev = kcache.device
        self.shape = shape
        self.T, self.prefix_len = T, prefix_len
        max_seq = kcache.shape[1]
        self.cfg = model_cfg(shape, max_seq, n_layers=len(model["layers"]))
        self._layers = (LayerWeights * max(1, len(model["layers"])))()
        for l, w in enumerate(model["layers"]):
            self._layers[l] = layer_weights(w)
        self.model = model    # packed (see pack_model)
        self.kcache, self.vcache = kcache, vcache
        self.mask = torch.zeros((T, 2), dtype=torch.int64, device=dev)
        self.pos = torch.zeros(T, dtype=torch.int32, device=dev)
        self.depth = torch.zeros(T, dtype=torch.int32, device=dev)
        self.resid = torch.zeros((T, shape.hidden), dtype=torch.float32, device=dev)
        self.logits = torch.zeros((T, shape.vocab), dtype=torch.float32, device=dev) if want_logits else None
        self.argmax = torch.zeros(T, dtype=torch.int32, device=dev)
        self.path = torch.zeros(T, dtype=torch.int32, device=dev)
        self.out_tokens = torch.zeros(T, dtype=torch.int32, device=dev)
        self.scalars = torch.zeros(4, dtype=torch.int32, device=dev)
        self.status = new_status(dev)
        self.ws = new_workspace(self.cfg, T, prefix_len, dev)
        self.hidden_in = hidden_in
        self.parent_stage = torch.zeros(T, dtype=torch.int32, device=dev)
        self.tokens_stage = torch.zeros(T, dtype=torch.int32, device=dev)
        a = ForwardArgs()
        a.cfg = C.pointer(self.cfg)
        a.layers = C.cast(self._layers, C.POINTER(LayerWeights))
        a.d_embed = _ptr(model.get("embed"))
        a.d_final_norm = _ptr(model["final_norm"])
        a.d_w_lm = _ptr(model["w_lm"])
        a.d_kcache, a.d_vcache = _ptr(kcache), _ptr(vcache)
        a.d_hidden_in = _ptr(hidden_in)
        a.T, a.prefix_len, a.compact = T, prefix_len, 1 if compact else 0
        a.d_mask, a.d_pos, a.d_depth, a.d_resid = _ptr(self.mask), _ptr(self.pos), _ptr(self.depth), _ptr(self.resid)
        a.d_logits, a.d_argmax, a.d_path = _ptr(self.logits), _ptr(self.argmax), _ptr(self.path)
        a.d_out_tokens, a.d_scalars = _ptr(self.out_tokens), _ptr(self.scalars)
        a.d_ws, a.ws_bytes, a.d_status = _ptr(self.ws), self.ws.numel(), _ptr(self.status)
        self.typical = None
        if typical is not None:
            self.typical = torch.zeros((3, T), dtype=torch.float32, device=dev)     # lse, entropy, candidate logits
            a.accept_mode = ACCEPT_TYPICAL
            a.inv_temperature, a.log_eps, a.log_delta = float(typical[0]), float(typical[1]), float(typical[2])
            a.d_typical = _ptr(self.typical)
        self.args = a

    def set_prefix_len(self, prefix_len: int):
        self.prefix_len = prefix_len
        self.args.prefix_len = prefix_len

    def run(self, d_parent, d_tokens):
        """cats_verify_forward on device inputs; asynchronous on the current stream."""
        _check(lib.cats_verify_forward(C.byref(self.args), _ptr(d_parent), _ptr(d_tokens), _stream()), "cats_verify_forward")

    def run_host(self, h_parent, h_tokens, h_scalars, h_out_tokens, h_path):
        """cats_verify_forward_host: host (ideally pinned) int32 tensors in and out; synchronises."""
        _check(lib.cats_verify_forward_host(C.byref(self.args), _ptr(h_parent), _ptr(h_tokens), _ptr(self.parent_stage),
                                            _ptr(self.tokens_stage), _ptr(h_scalars), _ptr(h_out_tokens), _ptr(h_path),
                                            _stream()), "cats_verify_forward_host")
