"""Algorithmic byte and flop counts of the tree-verification forward (what the method must move).

Every weight is read once per forward, the KV prefix once, the tree's K/V rows are written once and read
once; activations, split-K partial sums and logits are not counted.  The per-layer weight figure
(4 H^2 + 3 H F) * 2 bytes reproduces the paper's bytes-per-token baseline: 32 layers of a 7B model stream
12.95 GB per token (Table 4).
"""


def layer_weight_bytes(shape) -> int:
    H, F = shape.hidden, shape.ffn
    D = shape.n_heads * shape.head_dim
    return (3 * D * H + H * D + 3 * H * F) * 2


def lm_head_bytes(shape) -> int:
    return shape.vocab * shape.hidden * 2


def gemm_weight_bytes(shape) -> int:
    """Bytes streamed by all projection GEMMs of one forward (decoder layers + LM head)."""
    return shape.n_layers * layer_weight_bytes(shape) + lm_head_bytes(shape)


def gemm_launches(shape) -> int:
    """QKV, O, gate/up, down per layer, plus the LM head."""
    return 4 * shape.n_layers + 1


def kv_bytes(shape, prefix_len: int, T: int):
    row = shape.n_heads * shape.head_dim * 2
    read = shape.n_layers * 2 * (prefix_len + T) * row
    write = shape.n_layers * 2 * T * row
    return read, write


def forward_bytes(shape, prefix_len: int, T: int) -> int:
    read, write = kv_bytes(shape, prefix_len, T)
    gains = (2 * shape.n_layers + 1) * shape.hidden * 2
    embed_rows = T * shape.hidden * 2
    return gemm_weight_bytes(shape) + read + write + gains + embed_rows


def forward_flops(shape, prefix_len: int, T: int) -> int:
    params = gemm_weight_bytes(shape) // 2
    attn = shape.n_layers * 4 * T * (prefix_len + T) * shape.n_heads * shape.head_dim
    return 2 * T * params + attn


def attention_bytes(n_heads: int, head_dim: int, prefix_len: int, T: int) -> int:
    """Tree attention alone: K and V rows read once, q read and o written."""
    row = n_heads * head_dim * 2
    return 2 * (prefix_len + T) * row + 2 * T * row
