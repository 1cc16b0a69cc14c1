// C-ABI layer of libcats: argument checks, workspace layout, and the launch sequence of the
// tree-verification forward.  See include/cats.h for the contract of every entry point.
#include <cstring>

#include <nvtx3/nvToolsExt.h>

#include "cats_kernels.cuh"

namespace cats {

thread_local int g_launch_count = 0;
thread_local bool g_call_boundary = true;
int g_debug_attn_kernel = -1;
int g_debug_fault = 0;

namespace {


// Bring-up / measurement hook: bit i enables stage i of a decoder layer (0 norm1, 1 qkv, 2 attention,
// 3 o-proj, 4 norm2, 5 gate/up, 6 down).  All stages run by default.
unsigned g_stage_mask = 0x7f;
// Weights requested into L2 by the kernels that leave HBM idle (see WarmReq): {period, phase} per (issuing kernel,
// projection); period 0: none, -1: chosen from the size of the matrix.  Measured on the 7B forward (T = 64, 2.93 ms
// without): attention -> every third unit of gate/up 2.85 ms; plus the norm before QKV -> every fourth unit of QKV 2.80 ms;
// O or down projection units requested by the attention kernel, or gate/up units by the norm in front of it: no gain or
// a loss.  The budgets below are what HBM delivers while the issuing kernel runs.
//   [0] attention -> O   [1] attention -> gate/up   [2] attention -> down   [3] norm1 -> QKV   [4] norm2 -> gate/up
int g_warm[5][2] = {{0, 0}, {-1, 0}, {0, 0}, {-1, 0}, {0, 0}};
constexpr size_t kWarmBudget[5] = {0, (size_t)60 << 20, 0, (size_t)25 << 20, 0};
WarmReq warm_policy(int which, const void* ptr, size_t bytes) {
    int period = g_warm[which][0];
    if (period < 0) {
        period = kWarmBudget[which] ? (int)((bytes + kWarmBudget[which] / 2) / kWarmBudget[which]) : 0;
        if (period < 2 && kWarmBudget[which]) period = 2;
    }
    return warm_req(ptr, bytes, period, g_warm[which][1]);
}
inline bool stage_on(int i) { return (g_stage_mask >> i) & 1u; }

// One NVTX range per public call (visible in a timeline tool; a no-op when none is attached).
struct NvtxRange {
    explicit NvtxRange(const char* name) { nvtxRangePushA(name); }
    ~NvtxRange() { nvtxRangePop(); }
};

inline size_t align_up(size_t x, size_t a) { return (x + a - 1) / a * a; }

struct Workspace {
    uint8_t *xn, *o, *act;      // packed activation layout
    uint16_t* q;                // [T][D] row-major
    float* part;
    size_t part_stride;
    float2* rope;
    float *attn_o, *attn_ml;
    float* pmax;
    int32_t* pidx;
    float *psum, *ps1;          // per-tile softmax statistics of the LM head (typical acceptance)
    float* fix_part;
    int* fix_flags;
    float* scratch;             // [T][hidden] fp32
    int32_t* nodes;             // [CATS_MAX_TREE] clamped node list of a partial-tree forward
    size_t bytes;
};

int attn_split_bound(int nh) { int b = (148 + nh - 1) / nh; return b < 1 ? 1 : b; }   // clusters per head, upper bound

// Carves the workspace; with base == nullptr only the size is computed.
Workspace carve(const cats_model_cfg* c, int T, void* base) {
    Workspace w;
    size_t off = 0;
    auto take = [&](size_t bytes) { size_t o = off; off = align_up(off + bytes, 1024); return (uint8_t*)base + o; };
    const int D = c->n_heads * c->head_dim;
    const int tpad = (T + 15) / 16 * 16;
    auto packed = [&](int K) { return (size_t)((K + 63) / 64) * tpad * 128; };
    w.xn = take(packed(c->hidden));
    w.q = (uint16_t*)take((size_t)T * D * 2);
    w.o = take(packed(D));
    w.act = take(packed(c->ffn));
    w.part_stride = (size_t)T * c->hidden;
    w.part = (float*)take((size_t)kMaxPartSlots * w.part_stride * 4);
    w.rope = (float2*)take((size_t)T * (c->head_dim / 2) * sizeof(float2));
    size_t ns = attn_split_bound(c->n_heads);
    w.attn_o = (float*)take((size_t)c->n_heads * ns * tpad * c->head_dim * 4);
    w.attn_ml = (float*)take((size_t)c->n_heads * ns * tpad * 2 * 4);
    int vt = (c->vocab + 127) / 128;
    w.pmax = (float*)take((size_t)vt * 128 * 4);
    w.pidx = (int32_t*)take((size_t)vt * 128 * 4);
    w.psum = (float*)take((size_t)vt * 128 * 4);
    w.ps1 = (float*)take((size_t)vt * 128 * 4);
    w.fix_part = (float*)take((size_t)kFixSlots * tpad * 128 * 4);
    w.fix_flags = (int*)take((size_t)kFixSlots * sizeof(int));
    w.scratch = (float*)take((size_t)T * c->hidden * 4);
    w.nodes = (int32_t*)take((size_t)CATS_MAX_TREE * sizeof(int32_t));
    w.bytes = off;
    return w;
}

int check_cfg(const cats_model_cfg* c) {
    if (!c) return CATS_ERR_INVALID_ARG;
    if (c->hidden < 64 || c->n_heads < 1 || c->ffn < 8 || c->max_seq < 1) return CATS_ERR_INVALID_ARG;
    if (c->head_dim != 64 && c->head_dim != 128) return CATS_ERR_UNSUPPORTED;
    if (c->hidden % 64 || (c->n_heads * c->head_dim) % 64 || c->ffn % 8) return CATS_ERR_UNSUPPORTED;
    if (c->hidden > 16384) return CATS_ERR_UNSUPPORTED;
    return CATS_OK;
}

inline bool misaligned(const void* p, size_t a) { return (reinterpret_cast<uintptr_t>(p) % a) != 0; }

#define CATS_CUDA(expr)                              \
    do {                                             \
        cudaError_t e__ = (expr);                    \
        if (e__ != cudaSuccess) return CATS_ERR_CUDA; \
    } while (0)

// Split-K partial sums still to be folded into the residual stream by the next norm: n slices [T][hidden] fp32.
struct Pending {
    const float* part;
    int n;
    size_t stride;
};

// First half of a decoder layer over T rows: RMSNorm (folding `pend` into resid), QKV + RoPE + KV append, tree attention,
// O projection.  nodes == nullptr: the rows are the T tree nodes.  Else row t is tree node nodes[t] of a tree of T_tree
// nodes (mask and pos describe that whole tree): its K/V go to cache row P + nodes[t], it is rotated to pos[nodes[t]] and
// attends under mask row nodes[t]; the other tree rows are read from the cache.  copy_from: resid starts from this buffer.
// Returns the number of partial sums the O projection left in ws.part (> 0) or a negative status.
int layer_front(const cats_model_cfg* c, const cats_layer_weights* w, float* resid, const float* copy_from, void* kc, void* vc,
                const uint64_t* mask, const int32_t* pos, int T, int P, const Workspace& ws, Pending pend, int32_t* d_status,
                cudaStream_t st, const int32_t* nodes = nullptr, int T_tree = 0, bool rope_ready = false) {
    const int H = c->hidden, D = c->n_heads * c->head_dim;
    const int tpad = (T + 15) / 16 * 16;
    // rope_ready: an earlier layer of the same call has already left the rotary table of these rows in the workspace
    const WarmReq warm_qkv = warm_policy(3, w->wqkv, packed_weight_bytes(3, 0, D, H));
    if (stage_on(0))
        CATS_CUDA(launch_rmsnorm(resid, copy_from, pend.part, pend.n, pend.stride, w->attn_norm, T, H, c->rms_eps, ws.xn, pos,
                                 nodes, rope_ready ? nullptr : ws.rope, c->head_dim, c->rope_base, ws.fix_flags, kFixSlots, st,
                                 d_status, &warm_qkv));
    GemmProblem g = {};
    g.epi = EPI_QKV; g.T = T; g.K = H; g.n_out = D; g.n_mats = 3;
    g.W[0] = w->wqkv; g.X = ws.xn; g.fix_part = ws.fix_part; g.fix_flags = ws.fix_flags;
    g.q_out = ws.q; g.kcache = kc; g.vcache = vc; g.rope = ws.rope; g.head_dim = c->head_dim; g.prefix_len = P; g.kv_rows = nodes;
    g.d_status = d_status;
    if (stage_on(1)) CATS_CUDA(launch_gemm(g, st));

    AttnProblem a = {};
    a.q = ws.q; a.k = kc; a.v = vc; a.mask = mask; a.T = T; a.prefix_len = P; a.nh = c->n_heads; a.hd = c->head_dim;
    a.kv_stride = D; a.scale = 1.0f / sqrtf((float)c->head_dim); a.out = ws.o; a.out_packed_npad = tpad;
    a.part_o = ws.attn_o; a.part_ml = ws.attn_ml; a.d_status = d_status;
    a.nodes = nodes; a.T_tree = nodes ? T_tree : 0;
    attn_plan(a);
    a.warm[0] = warm_policy(0, w->wo, packed_weight_bytes(1, 0, H, D));
    a.warm[1] = warm_policy(1, w->w_gate_up, packed_weight_bytes(2, 1, c->ffn, H));
    a.warm[2] = warm_policy(2, w->w_down, packed_weight_bytes(1, 0, H, c->ffn));
    if (stage_on(2)) CATS_CUDA(launch_tree_attention(a, st));

    GemmProblem go = {};
    go.epi = EPI_PARTIAL; go.T = T; go.K = D; go.n_out = H; go.n_mats = 1; go.W[0] = w->wo; go.X = ws.o;
    go.fix_part = ws.fix_part; go.fix_flags = ws.fix_flags; go.part = ws.part; go.part_stride = ws.part_stride; go.d_status = d_status;
    const int pieces_o = gemm_plan(go).max_pieces;
    if (stage_on(3)) CATS_CUDA(launch_gemm(go, st));
    return pieces_o;
}

// Second half: RMSNorm (folding `pend`, the O projection's sums, into resid), gate/up + SwiGLU, down projection.
// Returns the number of partial sums the down projection left in ws.part (> 0) or a negative status.
int layer_back(const cats_model_cfg* c, const cats_layer_weights* w, float* resid, int T, const Workspace& ws, Pending pend,
               int32_t* d_status, cudaStream_t st) {
    const int H = c->hidden, F = c->ffn;
    GemmProblem ggu = {};
    ggu.epi = EPI_SWIGLU; ggu.T = T; ggu.K = H; ggu.n_out = F; ggu.n_mats = 2; ggu.W[0] = w->w_gate_up; ggu.X = ws.xn;
    ggu.fix_part = ws.fix_part; ggu.fix_flags = ws.fix_flags; ggu.act_out = ws.act; ggu.d_status = d_status;
    GemmProblem gd = {};
    gd.epi = EPI_PARTIAL; gd.T = T; gd.K = F; gd.n_out = H; gd.n_mats = 1; gd.W[0] = w->w_down; gd.X = ws.act;
    gd.fix_part = ws.fix_part; gd.fix_flags = ws.fix_flags; gd.part = ws.part; gd.part_stride = ws.part_stride; gd.d_status = d_status;
    const int pieces_d = gemm_plan(gd).max_pieces;
    const WarmReq warm_gu = warm_policy(4, w->w_gate_up, packed_weight_bytes(2, 1, F, H));
    if (stage_on(4))
        CATS_CUDA(launch_rmsnorm(resid, nullptr, pend.part, pend.n, pend.stride, w->mlp_norm, T, H, c->rms_eps, ws.xn, nullptr,
                                 nullptr, nullptr, c->head_dim, c->rope_base, nullptr, 0, st, d_status, &warm_gu));
    if (stage_on(5)) CATS_CUDA(launch_gemm(ggu, st));
    if (stage_on(6)) CATS_CUDA(launch_gemm(gd, st));
    return pieces_d;
}

// One whole decoder layer.  n_pending: split-K partial sums of the previous layer's down projection still to be folded
// into resid.  Returns the number of partial sums this layer's down projection left pending (> 0) or a negative status.
int layer_impl(const cats_model_cfg* c, const cats_layer_weights* w, float* resid, const float* copy_from, void* kc,
               void* vc, const uint64_t* mask, const int32_t* pos, int T, int P, const Workspace& ws, int n_pending,
               int32_t* d_status, cudaStream_t st, const int32_t* nodes = nullptr, int T_tree = 0, bool rope_ready = false) {
    const int pieces_o = layer_front(c, w, resid, copy_from, kc, vc, mask, pos, T, P, ws, Pending{ws.part, n_pending, ws.part_stride},
                                     d_status, st, nodes, T_tree, rope_ready);
    if (pieces_o < 0) return pieces_o;
    return layer_back(c, w, resid, T, ws, Pending{ws.part, pieces_o, ws.part_stride}, d_status, st);
}

// Typical acceptance: what the LM head must leave behind besides the argmax.
struct TypicalOut {
    const int32_t *parent, *tokens;   // [T] the tree
    float inv_temperature;
    float *lse, *entropy, *cand;      // [T] each
};

// vmax_out / idx_offset: a vocabulary shard also leaves every node's maximum and adds its first row to the indices.
int head_impl(const cats_model_cfg* c, const void* final_norm, const void* w_lm, float* resid, const float* copy_from,
              int T, Pending pend, float* logits, int32_t* amax, const Workspace& ws, int32_t* d_status, cudaStream_t st,
              const TypicalOut* ty = nullptr, float* vmax_out = nullptr, int idx_offset = 0) {
    const int H = c->hidden, V = c->vocab;
    CATS_CUDA(launch_rmsnorm(resid, copy_from, pend.part, pend.n, pend.stride, final_norm, T, H, c->rms_eps, ws.xn, nullptr,
                             nullptr, nullptr, c->head_dim, c->rope_base, ws.fix_flags, kFixSlots, st, d_status));
    GemmProblem g = {};
    g.epi = EPI_LMHEAD; g.T = T; g.K = H; g.n_out = V; g.n_mats = 1; g.W[0] = w_lm; g.X = ws.xn;
    g.fix_part = ws.fix_part; g.fix_flags = ws.fix_flags;
    g.logits = logits; g.pmax = ws.pmax; g.pidx = ws.pidx; g.d_status = d_status;
    if (ty) {
        g.psum = ws.psum; g.ps1 = ws.ps1; g.inv_temperature = ty->inv_temperature;
        g.tree_parent = ty->parent; g.tree_tokens = ty->tokens; g.cand = ty->cand;
    }
    CATS_CUDA(launch_gemm(g, st));
    if (ty)
        CATS_CUDA(launch_head_reduce(ws.pmax, ws.pidx, ws.psum, ws.ps1, (V + 127) / 128, 128, T, ty->inv_temperature, amax,
                                     ty->lse, ty->entropy, st));
    else
        CATS_CUDA(launch_argmax_reduce(ws.pmax, ws.pidx, (V + 127) / 128, 128, T, amax, vmax_out, idx_offset, st));
    return CATS_OK;
}

int check_tree_args(int T, int P) {
    if (T < 1 || T > CATS_MAX_TREE || P < 0) return CATS_ERR_INVALID_ARG;
    return CATS_OK;
}

}  // namespace
}  // namespace cats

using namespace cats;

extern "C" {

int cats_version(void) { return 100; }

const char* cats_status_string(int s) {
    switch (s) {
        case CATS_OK: return "ok";
        case CATS_ERR_INVALID_ARG: return "invalid argument";
        case CATS_ERR_BAD_TREE: return "malformed tree (parent array)";
        case CATS_ERR_UNSUPPORTED: return "unsupported shape";
        case CATS_ERR_WORKSPACE: return "workspace too small or misaligned";
        case CATS_ERR_CUDA: return "CUDA runtime error";
        case CATS_ERR_TIMEOUT: return "a bounded device-side wait expired";
        case CATS_ERR_UNIMPLEMENTED: return "not implemented";
        default: return "unknown status";
    }
}

int cats_last_launch_count(void) { return g_launch_count; }

/* Measurement and fault-injection hooks, declared in include/cats_debug.h. */
void cats_debug_stage_mask(unsigned mask) { g_stage_mask = mask & 0x7f; }
void cats_debug_attention_kernel(int which) { g_debug_attn_kernel = which < 0 ? -1 : (which > 2 ? 1 : which); }
void cats_debug_l2_warm(int which, int period, int phase) { if (which >= 0 && which < 5) { g_warm[which][0] = period; g_warm[which][1] = phase; } }
int cats_debug_timeline(int kernel, void* host, size_t bytes) {
    const bool clear = host == nullptr;
    cudaError_t e = cudaErrorInvalidValue;
    if (kernel == 0) e = timeline_gemm(host, bytes, clear);
    else if (kernel == 1) e = timeline_attn(host, bytes, clear);
    else if (kernel == 2) e = timeline_norm(host, bytes, clear);
    if (e == cudaErrorNotSupported) return CATS_ERR_UNSUPPORTED;
    return e == cudaSuccess ? CATS_OK : (e == cudaErrorInvalidValue ? CATS_ERR_INVALID_ARG : CATS_ERR_CUDA);
}
void cats_debug_inject_fault(int which) { g_debug_fault = (which == 1 || which == 2) ? which : 0; }
int cats_debug_wait_limit_ns(unsigned long long ns) {
    if (ns == 0) ns = kWaitLimitNs;
    if (set_wait_limit_gemm(ns) != cudaSuccess || set_wait_limit_attn(ns) != cudaSuccess || set_wait_limit_small(ns) != cudaSuccess)
        return CATS_ERR_CUDA;
    return CATS_OK;
}
int cats_debug_workspace_layout(const cats_model_cfg* cfg, int32_t T, size_t* out) {
    if (check_cfg(cfg) != CATS_OK || T < 1 || T > CATS_MAX_TREE || !out) return CATS_ERR_INVALID_ARG;
    Workspace w = carve(cfg, T, nullptr);
    out[0] = (size_t)((uint8_t*)w.xn - (uint8_t*)nullptr);
    out[1] = (size_t)((uint8_t*)w.q - (uint8_t*)nullptr);
    out[2] = (size_t)((uint8_t*)w.o - (uint8_t*)nullptr);
    out[3] = (size_t)((uint8_t*)w.act - (uint8_t*)nullptr);
    out[4] = (size_t)((uint8_t*)w.part - (uint8_t*)nullptr);
    out[5] = w.part_stride;
    GemmProblem g = {};
    g.epi = EPI_PARTIAL; g.T = T; g.K = cfg->n_heads * cfg->head_dim; g.n_out = cfg->hidden; g.n_mats = 1;
    out[6] = (size_t)gemm_plan(g).max_pieces;
    g.K = cfg->ffn;
    out[7] = (size_t)gemm_plan(g).max_pieces;
    return CATS_OK;
}

size_t cats_workspace_bytes(const cats_model_cfg* cfg, int32_t T, int32_t max_prefix) {
    (void)max_prefix;
    if (check_cfg(cfg) != CATS_OK || T < 1 || T > CATS_MAX_TREE) return 0;
    return carve(cfg, T, nullptr).bytes;
}

size_t cats_packed_weight_bytes(int32_t n_src, int32_t layout, int32_t rows, int32_t cols) {
    if (n_src < 1 || n_src > 3 || rows < 1 || cols < 1 || (layout != 0 && layout != 1) || (layout == 1 && n_src != 2)) return 0;
    return packed_weight_bytes(n_src, layout, rows, cols);
}

int cats_pack_weights(const void* const* d_src, int32_t n_src, int32_t layout, int32_t rows, int32_t cols, void* d_dst,
                      void* stream) {
    g_launch_count = 0;
    NvtxRange nvtx_range("cats_pack_weights");
    g_call_boundary = true;
    if (!d_src || !d_dst || cats_packed_weight_bytes(n_src, layout, rows, cols) == 0) return CATS_ERR_INVALID_ARG;
    for (int i = 0; i < n_src; ++i)
        if (!d_src[i] || misaligned(d_src[i], 16)) return CATS_ERR_INVALID_ARG;
    if (cols % 8 || misaligned(d_dst, 1024)) return CATS_ERR_INVALID_ARG;
    CATS_CUDA(launch_pack_weights(d_src, n_src, layout, rows, cols, d_dst, (cudaStream_t)stream));
    g_call_boundary = true;
    return CATS_OK;
}

int cats_build_tree_mask(const int32_t* d_parent, int32_t T, int32_t prefix_len, uint64_t* d_mask, int32_t* d_pos,
                         int32_t* d_depth, int32_t* d_status, void* stream) {
    g_launch_count = 0;
    NvtxRange nvtx_range("cats_build_tree_mask");
    g_call_boundary = true;
    if (!d_parent || !d_mask || !d_pos || !d_status) return CATS_ERR_INVALID_ARG;
    int rc = check_tree_args(T, prefix_len);
    if (rc) return rc;
    CATS_CUDA(launch_mask_pos(d_parent, T, prefix_len, d_mask, d_pos, d_depth, d_status, (cudaStream_t)stream));
    return CATS_OK;
}

int cats_embed_tokens(const void* d_embed, const int32_t* d_tokens, int32_t T, int32_t hidden, int32_t vocab, float* d_resid,
                      int32_t* d_status, void* stream) {
    g_launch_count = 0;
    NvtxRange nvtx_range("cats_embed_tokens");
    g_call_boundary = true;
    if (!d_embed || !d_tokens || !d_resid || !d_status) return CATS_ERR_INVALID_ARG;
    if (T < 1 || T > CATS_MAX_TREE || hidden < 8 || hidden % 8 || vocab < 1) return CATS_ERR_INVALID_ARG;
    if (misaligned(d_embed, 16) || misaligned(d_resid, 16)) return CATS_ERR_INVALID_ARG;
    CATS_CUDA(launch_embed(d_embed, d_tokens, T, hidden, vocab, d_resid, d_status, (cudaStream_t)stream));
    return CATS_OK;
}

int cats_verify_layer(const cats_model_cfg* cfg, const cats_layer_weights* w, float* d_resid, void* d_kcache, void* d_vcache,
                      const uint64_t* d_mask, const int32_t* d_pos, int32_t T, int32_t prefix_len, void* d_ws, size_t ws_bytes,
                      int32_t* d_status, void* stream) {
    g_launch_count = 0;
    NvtxRange nvtx_range("cats_verify_layer");
    g_call_boundary = true;
    int rc = check_cfg(cfg);
    if (rc) return rc;
    if (!w || !d_resid || !d_kcache || !d_vcache || !d_mask || !d_pos || !d_ws || !d_status) return CATS_ERR_INVALID_ARG;
    if (!w->attn_norm || !w->wqkv || !w->wo || !w->mlp_norm || !w->w_gate_up || !w->w_down) return CATS_ERR_INVALID_ARG;
    rc = check_tree_args(T, prefix_len);
    if (rc) return rc;
    if (prefix_len + T > cfg->max_seq) return CATS_ERR_INVALID_ARG;
    if (misaligned(d_ws, 1024)) return CATS_ERR_WORKSPACE;
    if (misaligned(d_resid, 16) || misaligned(d_kcache, 16) || misaligned(d_vcache, 16)) return CATS_ERR_INVALID_ARG;
    const void* ws_ptrs[] = {w->wqkv, w->wo, w->w_gate_up, w->w_down, w->attn_norm, w->mlp_norm};
    for (const void* p : ws_ptrs) if (misaligned(p, 16)) return CATS_ERR_INVALID_ARG;
    Workspace ws = carve(cfg, T, d_ws);
    if (ws.bytes > ws_bytes) return CATS_ERR_WORKSPACE;
    cudaStream_t st = (cudaStream_t)stream;
    int pending = layer_impl(cfg, w, d_resid, nullptr, d_kcache, d_vcache, d_mask, d_pos, T, prefix_len, ws, 0, d_status, st);
    if (pending < 0) return pending;
    if (stage_on(6))
        CATS_CUDA(launch_rmsnorm(d_resid, nullptr, ws.part, pending, ws.part_stride, nullptr, T, cfg->hidden, cfg->rms_eps, nullptr,
                             nullptr, nullptr, nullptr, cfg->head_dim, cfg->rope_base, nullptr, 0, st, d_status));
    return CATS_OK;
}

int cats_verify_layer_nodes(const cats_model_cfg* cfg, const cats_layer_weights* w, float* d_resid, void* d_kcache,
                            void* d_vcache, const uint64_t* d_mask, const int32_t* d_pos, const int32_t* d_nodes, int32_t m,
                            int32_t T, int32_t prefix_len, void* d_ws, size_t ws_bytes, int32_t* d_status, void* stream) {
    g_launch_count = 0;
    NvtxRange nvtx_range("cats_verify_layer_nodes");
    g_call_boundary = true;
    int rc = check_cfg(cfg);
    if (rc) return rc;
    if (!w || !d_resid || !d_kcache || !d_vcache || !d_mask || !d_pos || !d_nodes || !d_ws || !d_status) return CATS_ERR_INVALID_ARG;
    if (!w->attn_norm || !w->wqkv || !w->wo || !w->mlp_norm || !w->w_gate_up || !w->w_down) return CATS_ERR_INVALID_ARG;
    rc = check_tree_args(T, prefix_len);
    if (rc) return rc;
    if (m < 1 || m > T || prefix_len + T > cfg->max_seq) return CATS_ERR_INVALID_ARG;
    if (misaligned(d_ws, 1024)) return CATS_ERR_WORKSPACE;
    if (misaligned(d_resid, 16) || misaligned(d_kcache, 16) || misaligned(d_vcache, 16)) return CATS_ERR_INVALID_ARG;
    const void* ws_ptrs[] = {w->wqkv, w->wo, w->w_gate_up, w->w_down, w->attn_norm, w->mlp_norm};
    for (const void* p : ws_ptrs) if (misaligned(p, 16)) return CATS_ERR_INVALID_ARG;
    Workspace ws = carve(cfg, m, d_ws);
    if (ws.bytes > ws_bytes) return CATS_ERR_WORKSPACE;
    cudaStream_t st = (cudaStream_t)stream;
    CATS_CUDA(launch_check_nodes(d_nodes, m, T, ws.nodes, d_status, st));
    int pending = layer_impl(cfg, w, d_resid, nullptr, d_kcache, d_vcache, d_mask, d_pos, m, prefix_len, ws, 0, d_status, st,
                             ws.nodes, T);
    if (pending < 0) return pending;
    CATS_CUDA(launch_rmsnorm(d_resid, nullptr, ws.part, pending, ws.part_stride, nullptr, m, cfg->hidden, cfg->rms_eps, nullptr,
                             nullptr, nullptr, nullptr, cfg->head_dim, cfg->rope_base, nullptr, 0, st, d_status));
    return CATS_OK;
}

int cats_tree_attention(const void* d_q, const void* d_k, const void* d_v, const uint64_t* d_mask, int32_t T, int32_t prefix_len,
                        int32_t n_heads, int32_t head_dim, int64_t kv_row_stride_elems, float scale, void* d_out, void* d_ws,
                        size_t ws_bytes, int32_t* d_status, void* stream) {
    g_launch_count = 0;
    NvtxRange nvtx_range("cats_tree_attention");
    g_call_boundary = true;
    if (!d_q || !d_k || !d_v || !d_mask || !d_out || !d_status) return CATS_ERR_INVALID_ARG;
    int rc = check_tree_args(T, prefix_len);
    if (rc) return rc;
    if (n_heads < 1) return CATS_ERR_INVALID_ARG;
    if (head_dim != 64 && head_dim != 128) return CATS_ERR_UNSUPPORTED;
    if (kv_row_stride_elems < (int64_t)n_heads * head_dim || kv_row_stride_elems % 8) return CATS_ERR_INVALID_ARG;
    if (misaligned(d_q, 16) || misaligned(d_k, 16) || misaligned(d_v, 16) || misaligned(d_out, 4)) return CATS_ERR_INVALID_ARG;
    AttnProblem a = {};
    a.q = d_q; a.k = d_k; a.v = d_v; a.mask = d_mask; a.T = T; a.prefix_len = prefix_len; a.nh = n_heads; a.hd = head_dim;
    a.kv_stride = kv_row_stride_elems; a.scale = scale; a.out = d_out; a.d_status = d_status;
    size_t need = attn_plan(a);
    if (need > 0) {
        if (!d_ws || misaligned(d_ws, 16) || ws_bytes < need) return CATS_ERR_WORKSPACE;
        int tpad = (T + 15) / 16 * 16;
        a.part_o = (float*)d_ws;
        a.part_ml = a.part_o + (size_t)n_heads * a.n_splits * tpad * head_dim;
    }
    CATS_CUDA(launch_tree_attention(a, (cudaStream_t)stream));
    return CATS_OK;
}

int cats_lm_head_argmax(const cats_model_cfg* cfg, const void* d_final_norm, const void* d_w_lm, const float* d_resid, int32_t T,
                        float* d_logits, int32_t* d_argmax, void* d_ws, size_t ws_bytes, int32_t* d_status, void* stream) {
    g_launch_count = 0;
    NvtxRange nvtx_range("cats_lm_head_argmax");
    g_call_boundary = true;
    int rc = check_cfg(cfg);
    if (rc) return rc;
    if (!d_final_norm || !d_w_lm || !d_resid || !d_argmax || !d_ws || !d_status) return CATS_ERR_INVALID_ARG;
    if (T < 1 || T > CATS_MAX_TREE || cfg->vocab < 1) return CATS_ERR_INVALID_ARG;
    if (misaligned(d_ws, 1024)) return CATS_ERR_WORKSPACE;
    if (misaligned(d_resid, 16) || misaligned(d_w_lm, 16) || misaligned(d_final_norm, 16)) return CATS_ERR_INVALID_ARG;
    Workspace ws = carve(cfg, T, d_ws);
    if (ws.bytes > ws_bytes) return CATS_ERR_WORKSPACE;
    // the caller's residual is read-only here: normalise a copy held in the scratch area
    return head_impl(cfg, d_final_norm, d_w_lm, ws.scratch, d_resid, T, Pending{nullptr, 0, 0}, d_logits, d_argmax, ws, d_status,
                     (cudaStream_t)stream);
}

int cats_lm_head_typical(const cats_model_cfg* cfg, const void* d_final_norm, const void* d_w_lm, const float* d_resid,
                         const int32_t* d_parent, const int32_t* d_tokens, int32_t T, float inv_temperature, float* d_logits,
                         int32_t* d_argmax, float* d_lse, float* d_entropy, float* d_cand_logit, void* d_ws, size_t ws_bytes,
                         int32_t* d_status, void* stream) {
    g_launch_count = 0;
    NvtxRange nvtx_range("cats_lm_head_typical");
    g_call_boundary = true;
    int rc = check_cfg(cfg);
    if (rc) return rc;
    if (!d_final_norm || !d_w_lm || !d_resid || !d_parent || !d_tokens || !d_argmax || !d_lse || !d_entropy || !d_cand_logit ||
        !d_ws || !d_status)
        return CATS_ERR_INVALID_ARG;
    if (T < 1 || T > CATS_MAX_TREE || cfg->vocab < 1 || !(inv_temperature > 0.f) || !(inv_temperature < 1e6f)) return CATS_ERR_INVALID_ARG;
    if (misaligned(d_ws, 1024)) return CATS_ERR_WORKSPACE;
    if (misaligned(d_resid, 16) || misaligned(d_w_lm, 16) || misaligned(d_final_norm, 16)) return CATS_ERR_INVALID_ARG;
    Workspace ws = carve(cfg, T, d_ws);
    if (ws.bytes > ws_bytes) return CATS_ERR_WORKSPACE;
    cudaStream_t st = (cudaStream_t)stream;
    CATS_CUDA(cudaMemsetAsync(d_cand_logit, 0, (size_t)T * sizeof(float), st));
    g_call_boundary = true;   // the memset is not a kernel: the first kernel still takes full stream ordering
    TypicalOut ty = {d_parent, d_tokens, inv_temperature, d_lse, d_entropy, d_cand_logit};
    return head_impl(cfg, d_final_norm, d_w_lm, ws.scratch, d_resid, T, Pending{nullptr, 0, 0}, d_logits, d_argmax, ws, d_status, st, &ty);
}

int cats_accept_path_typical(const int32_t* d_parent, const int32_t* d_tokens, const int32_t* d_argmax, const float* d_cand_logit,
                             const float* d_lse, const float* d_entropy, int32_t T, float inv_temperature, float log_eps,
                             float log_delta, int32_t* d_path, int32_t* d_path_len, int32_t* d_out_tokens, int32_t* d_n_out,
                             int32_t* d_status, void* stream) {
    g_launch_count = 0;
    NvtxRange nvtx_range("cats_accept_path_typical");
    g_call_boundary = true;
    if (!d_parent || !d_tokens || !d_argmax || !d_cand_logit || !d_lse || !d_entropy || !d_path || !d_path_len || !d_out_tokens ||
        !d_n_out || !d_status)
        return CATS_ERR_INVALID_ARG;
    if (T < 1 || T > CATS_MAX_TREE || !(inv_temperature > 0.f)) return CATS_ERR_INVALID_ARG;
    CATS_CUDA(launch_walk_typical(d_parent, d_tokens, d_argmax, d_cand_logit, d_lse, d_entropy, T, inv_temperature, log_eps,
                                  log_delta, d_path, d_path_len, d_out_tokens, d_n_out, (cudaStream_t)stream));
    return CATS_OK;
}

int cats_accept_path(const int32_t* d_parent, const int32_t* d_tokens, const int32_t* d_argmax, int32_t T, int32_t* d_path,
                     int32_t* d_path_len, int32_t* d_out_tokens, int32_t* d_n_out, int32_t* d_status, void* stream) {
    g_launch_count = 0;
    NvtxRange nvtx_range("cats_accept_path");
    g_call_boundary = true;
    if (!d_parent || !d_tokens || !d_argmax || !d_path || !d_path_len || !d_out_tokens || !d_n_out || !d_status)
        return CATS_ERR_INVALID_ARG;
    if (T < 1 || T > CATS_MAX_TREE) return CATS_ERR_INVALID_ARG;
    CATS_CUDA(launch_walk(d_parent, d_tokens, d_argmax, T, d_path, d_path_len, d_out_tokens, d_n_out, d_status, (cudaStream_t)stream));
    return CATS_OK;
}

int cats_compact_kv(void* d_kcache, void* d_vcache, int32_t n_layers, int64_t layer_stride_elems, int64_t row_elems,
                    int32_t prefix_len, const int32_t* d_path, const int32_t* d_path_len, int32_t* d_new_len, int32_t* d_src_rows,
                    int32_t* d_dst_rows, int32_t* d_status, void* stream) {
    g_launch_count = 0;
    NvtxRange nvtx_range("cats_compact_kv");
    g_call_boundary = true;
    if (!d_kcache || !d_vcache || !d_path || !d_path_len || !d_status) return CATS_ERR_INVALID_ARG;
    if (n_layers < 1 || row_elems < 8 || row_elems % 8 || layer_stride_elems % 8 || prefix_len < 0) return CATS_ERR_INVALID_ARG;
    if (misaligned(d_kcache, 16) || misaligned(d_vcache, 16)) return CATS_ERR_INVALID_ARG;
    CATS_CUDA(launch_compact(d_kcache, d_vcache, n_layers, layer_stride_elems, row_elems, prefix_len, d_path, d_path_len,
                             d_new_len, d_src_rows, d_dst_rows, d_status, (cudaStream_t)stream));
    return CATS_OK;
}

/* ---- tensor-parallel halves (see cats.h) ---- */
static int tp_common_checks(const cats_model_cfg* cfg, const float* d_resid, int32_t T, void* d_ws, int32_t* d_status) {
    int rc = check_cfg(cfg);
    if (rc) return rc;
    if (!d_resid || !d_ws || !d_status) return CATS_ERR_INVALID_ARG;
    if (T < 1 || T > CATS_MAX_TREE) return CATS_ERR_INVALID_ARG;
    if (misaligned(d_ws, 1024)) return CATS_ERR_WORKSPACE;
    if (misaligned(d_resid, 16)) return CATS_ERR_INVALID_ARG;
    return CATS_OK;
}

int cats_tp_attention_half(const cats_model_cfg* cfg, const cats_layer_weights* w, float* d_resid, const float* d_pending,
                           void* d_kcache, void* d_vcache, const uint64_t* d_mask, const int32_t* d_pos, int32_t T,
                           int32_t prefix_len, float* d_partial_out, void* d_ws, size_t ws_bytes, int32_t* d_status, void* stream) {
    g_launch_count = 0;
    NvtxRange nvtx_range("cats_tp_attention_half");
    g_call_boundary = true;
    int rc = tp_common_checks(cfg, d_resid, T, d_ws, d_status);
    if (rc) return rc;
    if (!w || !w->attn_norm || !w->wqkv || !w->wo || !d_kcache || !d_vcache || !d_mask || !d_pos || !d_partial_out)
        return CATS_ERR_INVALID_ARG;
    if (prefix_len < 0 || prefix_len + T > cfg->max_seq) return CATS_ERR_INVALID_ARG;
    if (misaligned(d_partial_out, 16) || misaligned(d_pending, 16) || misaligned(d_kcache, 16) || misaligned(d_vcache, 16))
        return CATS_ERR_INVALID_ARG;
    Workspace ws = carve(cfg, T, d_ws);
    if (ws.bytes > ws_bytes) return CATS_ERR_WORKSPACE;
    cudaStream_t st = (cudaStream_t)stream;
    const size_t n = (size_t)T * cfg->hidden;
    const int pieces = layer_front(cfg, w, d_resid, nullptr, d_kcache, d_vcache, d_mask, d_pos, T, prefix_len, ws,
                                   Pending{d_pending, d_pending ? 1 : 0, n}, d_status, st);
    if (pieces < 0) return pieces;
    CATS_CUDA(launch_sum_parts(ws.part, pieces, ws.part_stride, n, d_partial_out, st));
    return CATS_OK;
}

int cats_tp_mlp_half(const cats_model_cfg* cfg, const cats_layer_weights* w, float* d_resid, const float* d_pending, int32_t T,
                     float* d_partial_out, void* d_ws, size_t ws_bytes, int32_t* d_status, void* stream) {
    g_launch_count = 0;
    NvtxRange nvtx_range("cats_tp_mlp_half");
    g_call_boundary = true;
    int rc = tp_common_checks(cfg, d_resid, T, d_ws, d_status);
    if (rc) return rc;
    if (!w || !w->mlp_norm || !w->w_gate_up || !w->w_down || !d_pending || !d_partial_out) return CATS_ERR_INVALID_ARG;
    if (misaligned(d_partial_out, 16) || misaligned(d_pending, 16)) return CATS_ERR_INVALID_ARG;
    Workspace ws = carve(cfg, T, d_ws);
    if (ws.bytes > ws_bytes) return CATS_ERR_WORKSPACE;
    cudaStream_t st = (cudaStream_t)stream;
    const size_t n = (size_t)T * cfg->hidden;
    // the stream-K fix-up flags of the gate/up projection must start at zero; the first half of the layer left them so
    const int pieces = layer_back(cfg, w, d_resid, T, ws, Pending{d_pending, 1, n}, d_status, st);
    if (pieces < 0) return pieces;
    CATS_CUDA(launch_sum_parts(ws.part, pieces, ws.part_stride, n, d_partial_out, st));
    return CATS_OK;
}

int cats_tp_lm_head_shard(const cats_model_cfg* cfg, const void* d_final_norm, const void* d_w_lm, float* d_resid,
                          const float* d_pending, int32_t T, int32_t vocab_offset, float* d_logits, float* d_max_out,
                          int32_t* d_argmax_out, void* d_ws, size_t ws_bytes, int32_t* d_status, void* stream) {
    g_launch_count = 0;
    NvtxRange nvtx_range("cats_tp_lm_head_shard");
    g_call_boundary = true;
    int rc = tp_common_checks(cfg, d_resid, T, d_ws, d_status);
    if (rc) return rc;
    if (!d_final_norm || !d_w_lm || !d_max_out || !d_argmax_out || cfg->vocab < 1 || vocab_offset < 0) return CATS_ERR_INVALID_ARG;
    if (misaligned(d_pending, 16) || misaligned(d_w_lm, 16) || misaligned(d_final_norm, 16)) return CATS_ERR_INVALID_ARG;
    Workspace ws = carve(cfg, T, d_ws);
    if (ws.bytes > ws_bytes) return CATS_ERR_WORKSPACE;
    const size_t n = (size_t)T * cfg->hidden;
    return head_impl(cfg, d_final_norm, d_w_lm, d_resid, nullptr, T, Pending{d_pending, d_pending ? 1 : 0, n}, d_logits, d_argmax_out,
                     ws, d_status, (cudaStream_t)stream, nullptr, d_max_out, vocab_offset);
}

int cats_tp_argmax_merge(const float* d_max, const int32_t* d_idx, int32_t n_shards, int32_t T, int32_t* d_argmax, void* stream) {
    g_launch_count = 0;
    NvtxRange nvtx_range("cats_tp_argmax_merge");
    g_call_boundary = true;
    if (!d_max || !d_idx || !d_argmax || n_shards < 1 || T < 1 || T > CATS_MAX_TREE) return CATS_ERR_INVALID_ARG;
    CATS_CUDA(launch_argmax_reduce(d_max, d_idx, n_shards, T, T, d_argmax, nullptr, 0, (cudaStream_t)stream));
    return CATS_OK;
}

int cats_verify_forward(const cats_forward_args* a, const int32_t* d_parent, const int32_t* d_tokens, void* stream) {
    g_launch_count = 0;
    NvtxRange nvtx_range("cats_verify_forward");
    g_call_boundary = true;
    if (!a || !d_parent || !d_tokens) return CATS_ERR_INVALID_ARG;
    const cats_model_cfg* c = a->cfg;
    int rc = check_cfg(c);
    if (rc) return rc;
    if (!a->layers || !a->d_final_norm || !a->d_w_lm || !a->d_kcache || !a->d_vcache || !a->d_mask || !a->d_pos || !a->d_resid ||
        !a->d_argmax || !a->d_path || !a->d_out_tokens || !a->d_scalars || !a->d_ws || !a->d_status)
        return CATS_ERR_INVALID_ARG;
    if (!a->d_hidden_in && !a->d_embed) return CATS_ERR_INVALID_ARG;
    rc = check_tree_args(a->T, a->prefix_len);
    if (rc) return rc;
    if (a->prefix_len + a->T > c->max_seq || c->n_layers < 0 || c->vocab < 1) return CATS_ERR_INVALID_ARG;
    if (a->accept_mode != CATS_ACCEPT_GREEDY && a->accept_mode != CATS_ACCEPT_TYPICAL) return CATS_ERR_INVALID_ARG;
    const bool typical = a->accept_mode == CATS_ACCEPT_TYPICAL;
    if (typical && (!a->d_typical || !(a->inv_temperature > 0.f) || !(a->inv_temperature < 1e6f))) return CATS_ERR_INVALID_ARG;
    if (misaligned(a->d_ws, 1024)) return CATS_ERR_WORKSPACE;
    if (misaligned(a->d_resid, 16) || misaligned(a->d_kcache, 16) || misaligned(a->d_vcache, 16)) return CATS_ERR_INVALID_ARG;
    Workspace ws = carve(c, a->T, a->d_ws);
    if (ws.bytes > a->ws_bytes) return CATS_ERR_WORKSPACE;
    cudaStream_t st = (cudaStream_t)stream;
    const int T = a->T, P = a->prefix_len;
    const size_t lstride = (size_t)c->max_seq * c->n_heads * c->head_dim;

    if (typical) CATS_CUDA(cudaMemsetAsync(a->d_typical + 2 * T, 0, (size_t)T * sizeof(float), st));   // candidate logits
    CATS_CUDA(launch_mask_pos(d_parent, T, P, a->d_mask, a->d_pos, a->d_depth, a->d_status, st));
    const float* copy_from = a->d_hidden_in;
    if (!copy_from) CATS_CUDA(launch_embed(a->d_embed, d_tokens, T, c->hidden, c->vocab, a->d_resid, a->d_status, st));
    int pending = 0;
    for (int l = 0; l < c->n_layers; ++l) {
        pending = layer_impl(c, &a->layers[l], a->d_resid, l == 0 ? copy_from : nullptr, (uint16_t*)a->d_kcache + l * lstride,
                             (uint16_t*)a->d_vcache + l * lstride, a->d_mask, a->d_pos, T, P, ws, pending, a->d_status, st,
                             nullptr, 0, /*rope_ready=*/l > 0 && stage_on(0));
        if (pending < 0) return pending;
    }
    TypicalOut ty = {d_parent, d_tokens, a->inv_temperature, a->d_typical, a->d_typical ? a->d_typical + T : nullptr,
                     a->d_typical ? a->d_typical + 2 * T : nullptr};
    rc = head_impl(c, a->d_final_norm, a->d_w_lm, a->d_resid, c->n_layers == 0 ? copy_from : nullptr, T,
                   Pending{ws.part, pending, ws.part_stride}, a->d_logits,
                   a->d_argmax, ws, a->d_status, st, typical ? &ty : nullptr);
    if (rc) return rc;
    if (typical)
        CATS_CUDA(launch_walk_typical(d_parent, d_tokens, a->d_argmax, ty.cand, ty.lse, ty.entropy, T, a->inv_temperature,
                                      a->log_eps, a->log_delta, a->d_path, a->d_scalars + 0, a->d_out_tokens, a->d_scalars + 1, st));
    else
        CATS_CUDA(launch_walk(d_parent, d_tokens, a->d_argmax, T, a->d_path, a->d_scalars + 0, a->d_out_tokens, a->d_scalars + 1, a->d_status, st));
    if (a->compact)
        CATS_CUDA(launch_compact(a->d_kcache, a->d_vcache, c->n_layers, (long long)lstride, (long long)c->n_heads * c->head_dim, P,
                                 a->d_path, a->d_scalars + 0, a->d_scalars + 2, nullptr, nullptr, a->d_status, st));
    return CATS_OK;
}

int cats_verify_forward_host(const cats_forward_args* a, const int32_t* h_parent, const int32_t* h_tokens, int32_t* d_parent_stage,
                             int32_t* d_tokens_stage, int32_t* h_scalars, int32_t* h_out_tokens, int32_t* h_path, void* stream) {
    if (!a || !h_parent || !h_tokens || !d_parent_stage || !d_tokens_stage || !h_scalars || !h_out_tokens || !h_path)
        return CATS_ERR_INVALID_ARG;
    if (a->T < 1 || a->T > CATS_MAX_TREE) return CATS_ERR_INVALID_ARG;
    cudaStream_t st = (cudaStream_t)stream;
    size_t nb = (size_t)a->T * sizeof(int32_t);
    CATS_CUDA(cudaMemcpyAsync(d_parent_stage, h_parent, nb, cudaMemcpyHostToDevice, st));
    CATS_CUDA(cudaMemcpyAsync(d_tokens_stage, h_tokens, nb, cudaMemcpyHostToDevice, st));
    int rc = cats_verify_forward(a, d_parent_stage, d_tokens_stage, stream);
    if (rc) return rc;
    CATS_CUDA(cudaMemcpyAsync(h_scalars, a->d_scalars, 3 * sizeof(int32_t), cudaMemcpyDeviceToHost, st));
    CATS_CUDA(cudaMemcpyAsync(h_scalars + 3, a->d_status, sizeof(int32_t), cudaMemcpyDeviceToHost, st));
    CATS_CUDA(cudaMemcpyAsync(h_out_tokens, a->d_out_tokens, nb, cudaMemcpyDeviceToHost, st));
    CATS_CUDA(cudaMemcpyAsync(h_path, a->d_path, nb, cudaMemcpyDeviceToHost, st));
    CATS_CUDA(cudaStreamSynchronize(st));
    return CATS_OK;
}

}  // extern "C"
