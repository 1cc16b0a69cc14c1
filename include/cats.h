/*
 * cats.h -- C ABI of libcats: the target model's tree-verification forward of
 * CATS-style self-speculative decoding (Algorithm 1, Stage 3 "Final
 * Verification", and the walk / roll-back that follow it), for NVIDIA B200
 * (sm_100a).
 *
 * One decoding cycle hands this library a draft token tree of T nodes
 * (1 <= T <= 128).  Node 0 is the root: the last committed token, whose K/V
 * rows are not yet in the cache.  parent[0] == -1 and 0 <= parent[i] < i.
 * The committed prefix has prefix_len tokens; their K/V rows are rows
 * [0, prefix_len) of every layer's cache.  Tree node i uses cache row
 * prefix_len + i until cats_compact_kv moves the accepted rows together.
 *
 * Conventions shared by every entry point
 *   - Pointers named d_* are DEVICE pointers; the caller owns every buffer.
 *     The library allocates no device memory.  The state it keeps is host-side
 *     and derived from arguments only: kernel attributes set once per process,
 *     a cache of up to 256 encoded tensor maps keyed by (pointer, shape) for
 *     the attention kernel, the per-device address of the scratch array of
 *     cats_tree_attention_static, and the switches of include/cats_debug.h
 *     (all at their defaults unless a test or a benchmark sets them).  No
 *     environment variable is read.
 *   - `stream` is a cudaStream_t passed as void*.  Calls are asynchronous,
 *     never synchronise and never copy to the host (except the *_host entry
 *     point, which says so).
 *   - Projection weights are bf16, handed over in the library's packed layout:
 *     cats_pack_weights converts nn.Linear matrices [out_features][in_features]
 *     (row-major) once, at load time.  Norm gains are bf16 [hidden].  16-bit
 *     tensors are raw bf16.
 *   - Return value: CATS_OK or a negative cats_status for problems the host
 *     can see (null pointer, T out of range, unsupported shape, short
 *     workspace, misaligned pointer); nothing is launched in that case.
 *   - Problems only the device can see (malformed parent array, a bounded wait
 *     that expired) are written with atomicMin into *d_status (an int32 the
 *     caller zeroes once); kernels then finish without touching memory out of
 *     bounds.  Kernels never trap.
 *   - Rounding contract: the residual stream and the logits are fp32; GEMM
 *     inputs (normalised hidden states, q, attention output, SwiGLU output)
 *     and the K/V cache are bf16, each rounded once from fp32; all sums,
 *     softmax, norms, SiLU and RoPE are computed in fp32.
 */
#ifndef CATS_H_
#define CATS_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

#define CATS_MAX_TREE 128

typedef enum {
    CATS_OK = 0,
    CATS_ERR_INVALID_ARG = -1,
    CATS_ERR_BAD_TREE = -2,
    CATS_ERR_UNSUPPORTED = -3,
    CATS_ERR_WORKSPACE = -4,
    CATS_ERR_CUDA = -5,
    CATS_ERR_TIMEOUT = -6,
    CATS_ERR_UNIMPLEMENTED = -7
} cats_status;

/* Decoder shape (LLaMA-2 / Vicuna family, the paper's target models): RMSNorm,
 * rotary embeddings with rotate-half pairing, multi-head attention with
 * n_kv_heads == n_heads, SwiGLU MLP, no biases.  head_dim must be 64 or 128,
 * hidden and n_heads*head_dim multiples of 64, ffn a multiple of 8. */
typedef struct {
    int32_t hidden, n_heads, head_dim, ffn, vocab, n_layers, max_seq;
    float rms_eps, rope_base;
} cats_model_cfg;

/* Device pointers to one layer's weights.  attn_norm, mlp_norm: bf16 [hidden].
 * wqkv: cats_pack_weights of {Wq, Wk, Wv} (layout 0, three matrices [n_heads*head_dim][hidden]);
 * wo: layout 0 of Wo [hidden][n_heads*head_dim]; w_gate_up: layout 1 of {W_gate, W_up}
 * ([ffn][hidden] each); w_down: layout 0 of W_down [hidden][ffn]. */
typedef struct {
    const void *attn_norm, *wqkv, *wo, *mlp_norm, *w_gate_up, *w_down;
} cats_layer_weights;

/* Weight packing.  The projections are bound by reading every weight once per
 * forward (Section 1: decoding is bound by weight movement; the byte model of
 * Eq. 3-4 counts exactly those bytes), so the library keeps each matrix as a sequence of
 * 16 KB chunks -- (128-row tile, 64-column block), already in the layout the
 * tensor cores read from shared memory -- that one SM can stream with plain
 * contiguous bulk copies.
 *   layout 0: n_src (1..3) matrices of identical shape [rows][cols] stacked, each
 *             padded to whole 128-row tiles.
 *   layout 1: n_src == 2 matrices (gate, up) interleaved as tiles of 64 + 64 rows,
 *             so that silu(gate)*up is computed inside one tile.
 * cols must be a multiple of 8; rows/cols beyond the matrix are stored as zeros.
 * d_src: HOST array of n_src device pointers (bf16, row-major, 16-byte aligned);
 * d_dst: device buffer of cats_packed_weight_bytes bytes, 1024-byte aligned.
 * cats_packed_weight_bytes returns 0 for invalid arguments. */
size_t cats_packed_weight_bytes(int32_t n_src, int32_t layout, int32_t rows, int32_t cols);
int cats_pack_weights(const void *const *d_src, int32_t n_src, int32_t layout, int32_t rows, int32_t cols,
                      void *d_dst, void *stream);

/* Ancestor mask, depth and position ids of the draft tree (the tree attention
 * mask of Fig. 4, which covers the main draft chain and the correction branches;
 * Algorithm 1, Stage 3, mask = T.tree_mask).
 *   d_parent [T] int32 in.  d_mask [T][2] uint64 out: bit j of row i (word
 *   j>>6, bit j&63) is set iff j == i or j is an ancestor of i.  d_pos [T]
 *   int32 out = prefix_len + depth.  d_depth [T] int32 out, may be NULL.
 * A malformed parent array sets *d_status = CATS_ERR_BAD_TREE; the outputs are
 * then zero masks and pos = prefix_len. */
int cats_build_tree_mask(const int32_t *d_parent, int32_t T, int32_t prefix_len, uint64_t *d_mask,
                         int32_t *d_pos, int32_t *d_depth, int32_t *d_status, void *stream);

/* Hidden states of the tree tokens from the embedding table (Algorithm 1,
 * T.hidden_states, for a forward that starts at layer 1).
 *   d_embed [vocab][hidden] bf16, d_tokens [T] int32 -> d_resid [T][hidden] fp32.
 * Token ids outside [0, vocab) set CATS_ERR_INVALID_ARG in *d_status and read row 0. */
int cats_embed_tokens(const void *d_embed, const int32_t *d_tokens, int32_t T, int32_t hidden, int32_t vocab,
                      float *d_resid, int32_t *d_status, void *stream);

/* Bytes of scratch cats_verify_layer / cats_lm_head_argmax / cats_tree_attention
 * need for trees of up to T nodes over prefixes of up to max_prefix tokens.
 * The workspace must be 1024-byte aligned. */
size_t cats_workspace_bytes(const cats_model_cfg *cfg, int32_t T, int32_t max_prefix);

/* One decoder layer over the T tree nodes under the tree mask (Algorithm 1,
 * Stage 3: H_tgt <- M_{L_SV+1:L_total}(T.hidden_states, mask, KV_M); Section
 * 3.2, final verification: all tree nodes go through the layers in one batch).
 *   d_resid [T][hidden] fp32, in/out: the residual stream.
 *   d_kcache/d_vcache: THIS layer's caches, bf16 [max_seq][n_heads*head_dim];
 *     rows [0,prefix_len) are read, rows prefix_len+i are written (k rotated).
 *   d_mask, d_pos: from cats_build_tree_mask.
 */
int cats_verify_layer(const cats_model_cfg *cfg, const cats_layer_weights *w, float *d_resid, void *d_kcache,
                      void *d_vcache, const uint64_t *d_mask, const int32_t *d_pos, int32_t T,
                      int32_t prefix_len, void *d_ws, size_t ws_bytes, int32_t *d_status, void *stream);

/* The same layer over a SUBSET of the tree (Algorithm 1, Stage 2: the
 * correction tokens are re-forwarded through layers 1..L_SV with the tree mask
 * applied, while the main-chain nodes already have their K/V in those
 * layers).
 *   d_nodes [m] int32, device: tree node indices, strictly ascending, in [0,T).
 *   d_resid [m][hidden] fp32 in/out: hidden states of those nodes only.
 *   d_mask [T][2], d_pos [T]: of the WHOLE tree (cats_build_tree_mask).
 *   Row j is rotated to d_pos[d_nodes[j]], its K/V are written to cache row
 *   prefix_len + d_nodes[j], and it attends to the prefix and to the tree rows
 *   mask row d_nodes[j] names.  Every cache row prefix_len..prefix_len+T-1
 *   that this call does not write is only read and must hold finite values
 *   (rows the mask hides are multiplied by a probability of exactly zero).
 *   The workspace is the one cats_workspace_bytes(cfg, T, ...) sizes.
 * A malformed node list sets *d_status = CATS_ERR_INVALID_ARG; the layer then
 * runs on the list clamped into [0,T) (no access leaves the buffers) and its
 * results are unspecified. */
int cats_verify_layer_nodes(const cats_model_cfg *cfg, const cats_layer_weights *w, float *d_resid, void *d_kcache,
                            void *d_vcache, const uint64_t *d_mask, const int32_t *d_pos, const int32_t *d_nodes,
                            int32_t m, int32_t T, int32_t prefix_len, void *d_ws, size_t ws_bytes,
                            int32_t *d_status, void *stream);

/* Tree-masked attention alone: node i of every head attends to cache rows
 * [0,prefix_len) and to row prefix_len+j iff bit j of d_mask[i] is set
 * (Fig. 4, tree attention mask; softmax(q.k * scale) v).
 *   d_q [T][n_heads][head_dim] bf16 (already rotated); d_k/d_v bf16 with
 *   kv_row_stride_elems elements between rows, head h at column h*head_dim;
 *   d_out [T][n_heads][head_dim] bf16. */
int cats_tree_attention(const void *d_q, const void *d_k, const void *d_v, const uint64_t *d_mask, int32_t T,
                        int32_t prefix_len, int32_t n_heads, int32_t head_dim, int64_t kv_row_stride_elems,
                        float scale, void *d_out, void *d_ws, size_t ws_bytes, int32_t *d_status, void *stream);

/* Bytes of scratch the library image itself carries on every GPU for the entry point below. */
#define CATS_STATIC_SCRATCH_BYTES (1u << 20)

/* cats_tree_attention for callers that cannot allocate.  (The paper has no counterpart: this is a
 * packaging variant of the same operation.)  Same arguments and result as cats_tree_attention, but
 * no workspace: the split-KV partial results go to a fixed CATS_STATIC_SCRATCH_BYTES array that is
 * part of the library and stays resident on every GPU that loads it, until the process exits.  It
 * is meant for code that has tensors but no way to get scratch memory at the call site: a plugin
 * that is handed buffers and no allocator, a region where touching the device allocator is not
 * allowed (someone else's stream capture), a real-time loop that must not call into the driver's
 * memory management.  The call performs no cudaMalloc/cudaFree and calls no allocating routine.
 *   - Scratch is needed only when one head is spread over several thread-block clusters (long
 *     prefixes with few heads): n_heads * clusters_per_head * ceil16(T) * (head_dim + 2) * 4 bytes.
 *     Problems needing more than the array holds (e.g. 14 heads x 128, T = 128, prefix 20000:
 *     1.9 MB) are refused with CATS_ERR_WORKSPACE and nothing is launched; use
 *     cats_tree_attention with a caller-owned workspace for those.
 *   - The first call on each device looks up the array's device address (with that device
 *     current) and caches it; make that first call outside any stream capture.
 *   - All calls on a device share the one array, and it keeps whatever the last call left in it.
 *     Nothing in it needs to start at zero (every slot that is read was written by the same call),
 *     but two calls whose kernels overlap on the GPU (different streams, or concurrent host
 *     threads) would overwrite each other's partial results: serialise them. */
int cats_tree_attention_static(const void *d_q, const void *d_k, const void *d_v, const uint64_t *d_mask, int32_t T,
                               int32_t prefix_len, int32_t n_heads, int32_t head_dim, int64_t kv_row_stride_elems,
                               float scale, void *d_out, int32_t *d_status, void *stream);

/* Final norm, LM head and per-node argmax (Algorithm 1: p_tgt <-
 * softmax(H(H_tgt)); greedy acceptance needs only argmax of the logits).
 *   d_logits [T][vocab] fp32 out, may be NULL.  d_argmax [T] int32 out: lowest
 *   vocabulary index attaining the maximum.  d_resid [T][hidden] fp32 in.
 *   d_w_lm: cats_pack_weights (layout 0) of the LM head [vocab][hidden]. */
int cats_lm_head_argmax(const cats_model_cfg *cfg, const void *d_final_norm, const void *d_w_lm,
                        const float *d_resid, int32_t T, float *d_logits, int32_t *d_argmax, void *d_ws,
                        size_t ws_bytes, int32_t *d_status, void *stream);

/* Greedy longest-accepted-path walk and bonus token (Algorithm 1, the walk
 * step of Stage 3: y_out and the bonus token).
 * A child is accepted iff its token equals d_argmax at its parent; among equal
 * sibling tokens the lowest node index wins.
 *   d_path [T] out: accepted node indices, d_path[0] = 0; *d_path_len >= 1.
 *   d_out_tokens [T] out: accepted draft tokens, then the bonus token;
 *   *d_n_out == *d_path_len. */
int cats_accept_path(const int32_t *d_parent, const int32_t *d_tokens, const int32_t *d_argmax, int32_t T,
                     int32_t *d_path, int32_t *d_path_len, int32_t *d_out_tokens, int32_t *d_n_out,
                     int32_t *d_status, void *stream);

/* Typical (relaxed) acceptance, the second criterion Acc that Algorithm 1
 * allows (the tables' relaxed setting at temperature 0.7), as the
 * cited Medusa work defines it: with p = softmax(logits / t) at the parent, a
 * child token x is acceptable iff  p(x) > min(eps, delta * exp(-H(p))).
 *
 * cats_lm_head_typical is cats_lm_head_argmax that also leaves, per node,
 *   d_lse [T] fp32        log sum_v exp(logits[n][v] / t)
 *   d_entropy [T] fp32    H(softmax(logits[n] / t))
 *   d_cand_logit [T] fp32 logits[parent[i]][tokens[i]] (0 for the root and for
 *                         tokens outside the vocabulary)
 * computed inside the LM-head kernel from its fp32 accumulators (the logits
 * need not be written).  d_parent, d_tokens: [T] int32, the tree.
 * inv_temperature = 1/t as fp32, 0 < 1/t < 1e6.
 *
 * cats_accept_path_typical walks the tree as Algorithm 1's loop does: from the
 * root, take the FIRST acceptable child in node order (the main draft token
 * before the correction at the same position), stop when there is none; the
 * bonus token is d_argmax at the last accepted node.  The verdict is taken in
 * the log domain in fp32, round to nearest, in this order:
 *     fma(d_cand_logit[i], inv_temperature, -d_lse[parent]) >
 *         min(log_eps, log_delta - d_entropy[parent])
 * so the caller passes log(eps) and log(delta) (the cited defaults: eps = 0.09,
 * delta = 0.3).  Outputs as cats_accept_path. */
int cats_lm_head_typical(const cats_model_cfg *cfg, const void *d_final_norm, const void *d_w_lm,
                         const float *d_resid, const int32_t *d_parent, const int32_t *d_tokens, int32_t T,
                         float inv_temperature, float *d_logits, int32_t *d_argmax, float *d_lse,
                         float *d_entropy, float *d_cand_logit, void *d_ws, size_t ws_bytes,
                         int32_t *d_status, void *stream);
int cats_accept_path_typical(const int32_t *d_parent, const int32_t *d_tokens, const int32_t *d_argmax,
                             const float *d_cand_logit, const float *d_lse, const float *d_entropy, int32_t T,
                             float inv_temperature, float log_eps, float log_delta, int32_t *d_path,
                             int32_t *d_path_len, int32_t *d_out_tokens, int32_t *d_n_out,
                             int32_t *d_status, void *stream);

/* KV roll-back along the accepted path (Algorithm 1, last step of the cycle):
 * for every layer, K and V, row
 * prefix_len + d_path[k] moves to row prefix_len + k, in place;
 * *d_new_len = prefix_len + *d_path_len.  Caches are 16-bit elements laid out
 * [n_layers][layer_stride_elems]; a row has row_elems elements (multiple of 8).
 * d_src_rows / d_dst_rows ([T] int32, may be NULL) receive the row indices. */
int cats_compact_kv(void *d_kcache, void *d_vcache, int32_t n_layers, int64_t layer_stride_elems,
                    int64_t row_elems, int32_t prefix_len, const int32_t *d_path, const int32_t *d_path_len,
                    int32_t *d_new_len, int32_t *d_src_rows, int32_t *d_dst_rows, int32_t *d_status,
                    void *stream);

enum { CATS_ACCEPT_GREEDY = 0, CATS_ACCEPT_TYPICAL = 1 };

/* Arguments of a whole verification forward (Stage 3 plus walk and roll-back). */
typedef struct {
    const cats_model_cfg *cfg;
    const cats_layer_weights *layers; /* HOST array of cfg->n_layers structs of device pointers */
    const void *d_embed;              /* [vocab][hidden] bf16; used when d_hidden_in == NULL */
    const void *d_final_norm;         /* [hidden] bf16 */
    const void *d_w_lm;               /* packed LM head (layout 0 of [vocab][hidden]) */
    void *d_kcache, *d_vcache;        /* [n_layers][max_seq][n_heads*head_dim] bf16 */
    const float *d_hidden_in;         /* [T][hidden] fp32 or NULL */
    int32_t T, prefix_len;
    int32_t compact;                  /* != 0: run cats_compact_kv at the end */
    /* device outputs, all caller-owned */
    uint64_t *d_mask;                 /* [T][2] */
    int32_t *d_pos, *d_depth;         /* [T] */
    float *d_resid;                   /* [T][hidden] */
    float *d_logits;                  /* [T][vocab] or NULL */
    int32_t *d_argmax, *d_path, *d_out_tokens; /* [T] */
    int32_t *d_scalars;               /* [4]: path_len, n_out, new_len, reserved */
    void *d_ws;
    size_t ws_bytes;
    int32_t *d_status;
    /* acceptance criterion of the walk */
    int32_t accept_mode;              /* CATS_ACCEPT_GREEDY or CATS_ACCEPT_TYPICAL */
    float inv_temperature;            /* typical: 1/t, log(eps), log(delta) as for cats_accept_path_typical */
    float log_eps, log_delta;
    float *d_typical;                 /* typical: [3][T] fp32 out: lse, entropy, candidate logits */
} cats_forward_args;

/* The whole path on device buffers: mask/pos, embedding (or caller's hidden
 * states), layers [0, n_layers), head + argmax, walk, compaction.  d_parent and
 * d_tokens are [T] int32 device arrays.  One asynchronous sequence of kernel
 * launches on `stream`, no host round trip. */
int cats_verify_forward(const cats_forward_args *a, const int32_t *d_parent, const int32_t *d_tokens,
                        void *stream);

/* Same, for HOST inputs and outputs: copies h_parent/h_tokens ([T] int32, host)
 * into d_parent_stage/d_tokens_stage, runs cats_verify_forward, copies back
 * h_scalars[4] (path_len, n_out, new_len, status), h_out_tokens[T] and
 * h_path[T], and synchronises the stream before returning. */
int cats_verify_forward_host(const cats_forward_args *a, const int32_t *h_parent, const int32_t *h_tokens,
                             int32_t *d_parent_stage, int32_t *d_tokens_stage, int32_t *h_scalars,
                             int32_t *h_out_tokens, int32_t *h_path, void *stream);

/* ---- Tensor-parallel verification over R GPUs -------------------------------
 * (The paper runs on an 8-GPU server, Section 4 "Experimental setup", but gives
 * no mechanism; this split is this library's.)  Rank r holds the attention
 * heads [r*nh/R, (r+1)*nh/R) -- the matching rows of Wq, Wk, Wv, columns of Wo
 * and its own slice [max_seq][nh/R*hd] of every layer's K/V cache -- and the
 * MLP rows [r*F/R, (r+1)*F/R) of W_gate, W_up (columns of W_down); norm gains
 * and the residual stream are replicated.  A layer is two calls per rank, each
 * leaving this rank's CONTRIBUTION to the residual stream as one [T][hidden]
 * fp32 tensor that the caller sums over the ranks (one all-reduce, e.g. NCCL
 * over NVLink) and hands to the next call as d_pending, where the norm folds it
 * into the rank's copy of the residual stream:
 *
 *   cats_tp_attention_half: resid += pending (NULL for the first layer);
 *       norm, QKV + RoPE + KV append, tree attention, O projection of this
 *       rank's heads -> d_partial_out
 *   cats_tp_mlp_half:       resid += pending (the all-reduced attention sums);
 *       norm, gate/up + SwiGLU, down projection of this rank's rows
 *       -> d_partial_out
 *
 * cfg is the SHARD's shape: hidden as in the full model, n_heads = nh/R,
 * ffn = F/R, vocab = V/R (head_dim 64 or 128, n_heads*head_dim a multiple of
 * 64, ffn a multiple of 8); w holds the packed shard matrices.  All ranks see
 * identical residual streams as long as the all-reduce delivers identical sums.
 *
 * cats_tp_lm_head_shard: resid += pending (the last layer's all-reduced MLP
 * sums); final norm; logits of vocabulary rows [vocab_offset, vocab_offset +
 * cfg->vocab); d_max_out [T] fp32 = this shard's maximum per node, d_argmax_out
 * [T] = its lowest GLOBAL index; d_logits [T][cfg->vocab] optional.  The caller
 * gathers (max, index) of all shards as [R][T] arrays; cats_tp_argmax_merge picks
 * per node the greatest maximum, lowest index on ties (= the argmax of the
 * unsplit head).  Walk and compaction then run on every rank as usual, the
 * compaction on the rank's cache slice (row_elems = nh/R*hd). */
int cats_tp_attention_half(const cats_model_cfg *cfg, const cats_layer_weights *w, float *d_resid, const float *d_pending,
                           void *d_kcache, void *d_vcache, const uint64_t *d_mask, const int32_t *d_pos, int32_t T,
                           int32_t prefix_len, float *d_partial_out, void *d_ws, size_t ws_bytes, int32_t *d_status,
                           void *stream);
int cats_tp_mlp_half(const cats_model_cfg *cfg, const cats_layer_weights *w, float *d_resid, const float *d_pending, int32_t T,
                     float *d_partial_out, void *d_ws, size_t ws_bytes, int32_t *d_status, void *stream);
int cats_tp_lm_head_shard(const cats_model_cfg *cfg, const void *d_final_norm, const void *d_w_lm, float *d_resid,
                          const float *d_pending, int32_t T, int32_t vocab_offset, float *d_logits, float *d_max_out,
                          int32_t *d_argmax_out, void *d_ws, size_t ws_bytes, int32_t *d_status, void *stream);
int cats_tp_argmax_merge(const float *d_max, const int32_t *d_idx, int32_t n_shards, int32_t T, int32_t *d_argmax,
                         void *stream);

/* Number of kernel launches the last call of this thread issued (for reports). */
int cats_last_launch_count(void);

const char *cats_status_string(int status);
int cats_version(void);

#ifdef __cplusplus
}
#endif
#endif /* CATS_H_ */
