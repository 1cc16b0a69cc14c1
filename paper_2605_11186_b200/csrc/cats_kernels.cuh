// Internal interface between the C-ABI layer (cats_api.cu) and the kernel files.
#pragma once

#include <cuda.h>

#include "cats_common.cuh"

namespace cats {

// Counts launches issued by the calling thread (reported through cats_last_launch_count).
extern thread_local int g_launch_count;
// Set at the top of every public entry point: the first kernel of a call is launched with full
// stream ordering, so nothing a call does before its griddepcontrol.wait (weight and KV-prefix
// prefetch) can overlap work issued by earlier calls.
extern thread_local bool g_call_boundary;

// Measurement / fault-injection state set through the cats_debug_* hooks (include/cats_debug.h); process-wide.
extern int g_debug_attn_kernel;   // -1: attention kernel chosen by shape; 0: mma.sync kernel; 1: tcgen05 kernel; 2: tcgen05 kernel,
                                  // two softmax threads per query row instead of four
extern int g_debug_fault;         // 0: none; 1: a helper CTA of a projection never publishes; 2: the attention loader drops Q
cudaError_t set_wait_limit_gemm(unsigned long long ns);
cudaError_t set_wait_limit_attn(unsigned long long ns);
cudaError_t set_wait_limit_small(unsigned long long ns);

// Launch with programmatic stream serialization: the kernel may start while its predecessor in the
// stream is still draining; every kernel calls griddepcontrol.wait before touching dependent data.
template <typename... KArgs, typename... Args>
inline cudaError_t launch_pdl(void (*kernel)(KArgs...), dim3 grid, dim3 block, size_t smem, cudaStream_t st, Args... args) {
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = grid;
    cfg.blockDim = block;
    cfg.dynamicSmemBytes = smem;
    cfg.stream = st;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr;
    cfg.numAttrs = g_call_boundary ? 0 : 1;
    g_call_boundary = false;
    ++g_launch_count;
    return cudaLaunchKernelEx(&cfg, kernel, static_cast<KArgs>(args)...);
}

// ---- small kernels ---------------------------------------------------------------------------
cudaError_t launch_mask_pos(const int32_t* parent, int T, int prefix_len, uint64_t* mask, int32_t* pos, int32_t* depth,
                            int32_t* d_status, cudaStream_t st);
cudaError_t launch_embed(const void* E, const int32_t* tokens, int T, int H, int vocab, float* resid, int32_t* d_status,
                         cudaStream_t st);
cudaError_t launch_rmsnorm(float* resid, const float* copy_from, const float* part, int n_part, size_t part_stride,
                           const void* gain, int T, int H, float eps, void* xn_packed, const int32_t* pos, const int32_t* nodes,
                           float2* rope, int hd, float rope_base, int* zero_flags, int n_flags, cudaStream_t st,
                           int32_t* d_status = nullptr, const WarmReq* warm = nullptr);   // warm: see WarmReq (register kernel only)
// Time lines (builds with -DCATS_TIMELINE; cudaErrorNotSupported otherwise): every launch of the kernel writes a slot of
// [kTlCtas][kTlStamps] 64-bit words, the stamps being %globaltimer values at points listed beside each kernel.
cudaError_t timeline_gemm(void* host, size_t bytes, bool clear);    // 512 slots
cudaError_t timeline_attn(void* host, size_t bytes, bool clear);    // 128 slots (tcgen05 kernel)
cudaError_t timeline_norm(void* host, size_t bytes, bool clear);    // 256 slots (k_rmsnorm_reg)
// Checks a partial-tree node list (strictly ascending, inside [0, T)) and writes a copy clamped into range.
cudaError_t launch_check_nodes(const int32_t* nodes, int m, int T, int32_t* clamped, int32_t* d_status, cudaStream_t st);
cudaError_t launch_argmax_reduce(const float* pmax, const int32_t* pidx, int n_tiles, int t_stride, int T, int32_t* amax,
                                 float* vmax, int idx_offset, cudaStream_t st);
// out[i] = sum over the n_part slices part[s * part_stride + i], i < n (n and part_stride multiples of 4).
cudaError_t launch_sum_parts(const float* part, int n_part, size_t part_stride, size_t n, float* out, cudaStream_t st);
// The same reduction plus the merge of the per-tile softmax statistics: lse[n] = log sum_v exp(logit/t),
// entropy[n] = H(softmax(logit/t)).
cudaError_t launch_head_reduce(const float* pmax, const int32_t* pidx, const float* psum, const float* ps1, int n_tiles,
                               int t_stride, int T, float inv_temperature, int32_t* amax, float* lse, float* entropy,
                               cudaStream_t st);
cudaError_t launch_walk_typical(const int32_t* parent, const int32_t* tokens, const int32_t* amax, const float* cand,
                                const float* lse, const float* entropy, int T, float inv_temperature, float log_eps,
                                float log_delta, int32_t* path, int32_t* path_len, int32_t* out_tokens, int32_t* n_out,
                                cudaStream_t st);
cudaError_t launch_walk(const int32_t* parent, const int32_t* tokens, const int32_t* amax, int T, int32_t* path,
                        int32_t* path_len, int32_t* out_tokens, int32_t* n_out, int32_t* d_status, cudaStream_t st);
cudaError_t launch_compact(void* kc, void* vc, int n_layers, long long layer_stride, long long row_elems, int prefix_len,
                           const int32_t* path, const int32_t* path_len, int32_t* new_len, int32_t* src_rows,
                           int32_t* dst_rows, int32_t* d_status, cudaStream_t st);

// ---- skinny weight-streaming GEMM ----------------------------------------------------------------
// Y^T[n_out, T] = W[n_out, K] * X^T[K, T]: weight rows are the MMA's M dimension (128 per tile), the
// tree nodes its N dimension (T padded to a multiple of 16).  W is packed by launch_pack_weights, X is
// in the packed activation layout (packed_act_offset).
enum GemmEpilogue : int {
    EPI_PARTIAL = 0,  // fp32 split-K partial sums  part[piece][t][n_out]
    EPI_QKV = 1,      // RoPE on q and k, bf16 q out, k/v appended to the cache rows prefix_len + t
    EPI_SWIGLU = 2,   // tile = 64 gate rows + 64 up rows -> a[t][f] = bf16(silu(gate) * up), packed layout
    EPI_LMHEAD = 3    // optional fp32 logits, per-tile (max, lowest index) per node
};

constexpr int kGemmCtas = 148;      // one persistent CTA per SM
constexpr int kFixSlots = 2 * kGemmCtas;   // partial-tile slots: one per CTA, or two per tile when helpers are used
constexpr int kMaxPartSlots = 8;    // partial-sum slots of EPI_PARTIAL

struct GemmProblem {
    int epi;
    int T;            // tree nodes
    int K;            // reduction length (in_features)
    int n_out;        // output features of ONE weight matrix (QKV: n_heads*head_dim; SwiGLU: ffn)
    int n_mats;       // 1, or 3 for QKV, or 2 for SwiGLU
    const void* W[3]; // W[0]: packed weights (all matrices of the problem in one buffer)
    const void* X;    // packed activations
    float* fix_part;  // [kFixSlots][n_pad][128] fp32: partial tiles of tiles shared by several CTAs
    int* fix_flags;   // [kFixSlots], zero between launches
    // epilogue operands
    float* part;           // EPI_PARTIAL: [pieces][T][n_out]
    size_t part_stride;    //   elements between slots
    void* q_out;           // EPI_QKV: [T][n_out] bf16
    void* kcache;          //   [max_seq][n_out] bf16 (this layer)
    void* vcache;
    const float2* rope;    //   [T][head_dim/2] (cos, sin)
    int head_dim;
    int prefix_len;
    const int32_t* kv_rows; //   null: node t goes to cache row prefix_len + t; else to prefix_len + kv_rows[t]
    void* act_out;         // EPI_SWIGLU: packed activations, ceil(n_out/64) K blocks
    float* logits;         // EPI_LMHEAD: [T][n_out] fp32 or null
    float* pmax;           //   [n_tiles][128]
    int32_t* pidx;
    float* psum;           //   optional (typical acceptance): per-tile sum of exp((logit - tile max) / t) ...
    float* ps1;            //   ... and sum of exp(..) * (logit - tile max), [n_tiles][128] each
    float inv_temperature;
    const int32_t* tree_parent;   //   [T] parent of every tree node
    const int32_t* tree_tokens;   //   [T] token of every tree node
    float* cand;           //   [T] out: logits[parent[i]][tokens[i]]
    int32_t* d_status;
};

struct GemmPlan {
    int units_per_cta;   // (tile, K block) pairs per CTA, contiguous
    int n_ctas;
    int max_pieces;      // EPI_PARTIAL: number of partial-sum slots the following reduction must fold
    int split_s;         // > 0: every tile is cut into this many aligned pieces (CTA = tile * split_s + piece)
    int head_units;      // > 0: one owner CTA per tile runs this many K units, helper CTAs share the rest
    int help_upc;        //      units per helper CTA
};

// Number of 128-row tiles the problem has (SwiGLU: tiles of 64 gate + 64 up rows).
int gemm_num_tiles(const GemmProblem& p);
GemmPlan gemm_plan(const GemmProblem& p);
cudaError_t launch_gemm(const GemmProblem& p, cudaStream_t st);
size_t packed_weight_bytes(int n_src, int layout, int rows, int cols);
cudaError_t launch_pack_weights(const void* const* src, int n_src, int layout, int rows, int cols, void* dst, cudaStream_t st);

// ---- tree attention --------------------------------------------------------------------------------
struct AttnProblem {
    const void* q;      // [T][nh][hd] bf16
    const void* k;      // rows of kv_stride elements, head h at h*hd
    const void* v;
    const uint64_t* mask;
    int T, prefix_len, nh, hd;   // T: query rows
    int T_tree;                  // tree rows in the cache after the prefix (0: the same as T)
    const int32_t* nodes;        // null: query t is tree node t; else query t is tree node nodes[t] (its mask row)
    long long kv_stride;
    float scale;
    void* out;          // [T][nh][hd] bf16, or the packed activation layout if out_packed_npad > 0
    int out_packed_npad;
    float* part_o;      // [nh][n_splits][T_pad][hd] fp32 (n_splits > 1 only)
    float* part_ml;     // [nh][n_splits][T_pad][2]
    int n_splits;       // filled by attn_plan: clusters per head (> 1 only for long prefixes with few heads)
    int cluster;        //   CTAs per cluster
    int rows_per_split; //   cache rows per CTA (multiple of 16)
    int qsplit;         //   > 0: CTAs per head that split the query tiles instead (every CTA reads all cache rows)
    int mt_per_cta;     //   query tiles per CTA in that case
    int use_tc;         //   1: the tcgen05 kernel (head_dim 128)
    int32_t* d_status;
    WarmReq warm[3];    // weights of the projections that follow, to be requested into L2 (tcgen05 kernel, one-block shares)
};
// Chooses the KV split; returns bytes of partial storage needed.
size_t attn_plan(AttnProblem& p);
cudaError_t launch_tree_attention(const AttnProblem& p, cudaStream_t st);

}  // namespace cats
