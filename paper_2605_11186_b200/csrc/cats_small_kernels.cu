// Latency-bound kernels of the tree-verification forward: ancestor mask / position ids, embedding
// gather, RMSNorm (fused with the split-K reduction of the preceding projection and with the RoPE
// table), argmax reduction, the greedy accepted-path walk and KV compaction.
#include "cats_kernels.cuh"

namespace cats {

// ---------------------------------------------------------------------------------------------
// Ancestor mask, depth, position ids.  One CTA of 128 threads; thread i walks from node i to the
// root, OR-ing one bit per node met.  A malformed parent array (parent[0] != -1, parent[i] outside
// [0, i)) reports CATS_ERR_BAD_TREE and produces zero masks; the walk is bounded by T steps.
// ---------------------------------------------------------------------------------------------
__global__ void __launch_bounds__(kMaxTree) k_mask_pos(const int32_t* __restrict__ parent, int T, int prefix_len,
                                                        uint64_t* __restrict__ mask, int32_t* __restrict__ pos,
                                                        int32_t* __restrict__ depth, int32_t* d_status) {
    __shared__ int32_t sp[kMaxTree];
    __shared__ int bad;
    pdl_launch_dependents();
    pdl_wait();
    int i = threadIdx.x;
    if (i == 0) bad = 0;
    __syncthreads();
    if (i < T) {
        int p = parent[i];
        sp[i] = p;
        if ((i == 0 && p != -1) || (i > 0 && (p < 0 || p >= i))) bad = 1;
    }
    __syncthreads();
    if (i >= T) return;
    if (bad) {
        if (i == 0) report(d_status, CATS_ERR_BAD_TREE);
        mask[2 * i] = 0;
        mask[2 * i + 1] = 0;
        pos[i] = prefix_len;
        if (depth) depth[i] = 0;
        return;
    }
    uint64_t m0 = 0, m1 = 0;
    int d = 0, j = i;
    for (int step = 0; step < T && j >= 0; ++step) {
        if (j < 64) m0 |= 1ull << j; else m1 |= 1ull << (j - 64);
        j = sp[j];
        if (j >= 0) ++d;
    }
    mask[2 * i] = m0;
    mask[2 * i + 1] = m1;
    pos[i] = prefix_len + d;
    if (depth) depth[i] = d;
}

// ---------------------------------------------------------------------------------------------
// Embedding gather: resid[t][:] = float(E[tokens[t]][:]).  One CTA per token.
// ---------------------------------------------------------------------------------------------
__global__ void __launch_bounds__(256) k_embed(const uint16_t* __restrict__ E, const int32_t* __restrict__ tokens, int H,
                                               int vocab, float* __restrict__ resid, int32_t* d_status) {
    pdl_launch_dependents();
    pdl_wait();
    int t = blockIdx.x;
    int tok = tokens[t];
    if (tok < 0 || tok >= vocab) {
        if (threadIdx.x == 0) report(d_status, CATS_ERR_INVALID_ARG);
        tok = 0;
    }
    const uint4* src = reinterpret_cast<const uint4*>(E + (size_t)tok * H);
    float4* dst = reinterpret_cast<float4*>(resid + (size_t)t * H);
    for (int c = threadIdx.x; c < H / 8; c += blockDim.x) {
        uint4 v = src[c];
        uint32_t w[4] = {v.x, v.y, v.z, v.w};
        float f[8];
#pragma unroll
        for (int q = 0; q < 4; ++q) {
            f[2 * q] = __uint_as_float(w[q] << 16);
            f[2 * q + 1] = __uint_as_float(w[q] & 0xFFFF0000u);
        }
        dst[2 * c] = make_float4(f[0], f[1], f[2], f[3]);
        dst[2 * c + 1] = make_float4(f[4], f[5], f[6], f[7]);
    }
}

// ---------------------------------------------------------------------------------------------
// RMSNorm, one CTA per tree node.  Before normalising it folds n_part split-K partial sums of the
// preceding projection into the fp32 residual stream (fixed order, so results are reproducible):
//   resid[t] (+)= part[0][t] + part[1][t] + ...;   xn[t] = bf16(g * resid[t] * rsqrt(mean(resid[t]^2) + eps)).
// xn is written in the packed activation layout the GEMM reads (n_pad rows per K block).
// copy_from (optional): resid[t] starts from copy_from[t] instead of its own contents.
// rope (optional): also fills the rotary table rope[t][i] = (cos, sin)(pos[t] * base^(-2i/hd)), i < hd/2,
// evaluated in fp64 so that large positions lose no accuracy.
// zero_flags (optional): CTA 0 clears the GEMM's stream-K flags (they are clear after every
// successful launch; this guards against an uninitialised workspace).
// ---------------------------------------------------------------------------------------------
__global__ void __launch_bounds__(256) k_rmsnorm(float* __restrict__ resid, const float* __restrict__ copy_from,
                                                 const float* __restrict__ part, int n_part, size_t part_stride,
                                                 const uint16_t* __restrict__ gain, int H, float eps,
                                                 uint8_t* __restrict__ xn, int n_pad, const int32_t* __restrict__ pos,
                                                 const int32_t* __restrict__ nodes, float2* __restrict__ rope, int hd, float rope_base, int* zero_flags,
                                                 int n_flags) {
    extern __shared__ float srow[];  // H floats
    __shared__ float red[8];
    pdl_launch_dependents();
    int t = blockIdx.x;
    pdl_wait();
    if (zero_flags != nullptr && t == 0)
        for (int i = threadIdx.x; i < n_flags; i += blockDim.x) zero_flags[i] = 0;
    if (rope != nullptr) {
        int half = hd / 2;
        int p = pos[nodes != nullptr ? nodes[t] : t];   // row t holds tree node nodes[t]
        for (int i = threadIdx.x; i < half; i += blockDim.x) {
            double inv_freq = pow((double)rope_base, -2.0 * (double)i / (double)hd);
            double s, c;
            sincos((double)p * inv_freq, &s, &c);
            rope[(size_t)t * half + i] = make_float2((float)c, (float)s);
        }
    }
    const float4* r4 = reinterpret_cast<const float4*>((copy_from ? copy_from : resid) + (size_t)t * H);
    float ss = 0.f;
    for (int c = threadIdx.x; c < H / 4; c += blockDim.x) {
        float4 v = r4[c];
        // all partial-sum loads of this column group are issued before the first add (their latencies overlap);
        // the adds keep slot order, so the result does not depend on how the loads return
        float4 pv[kMaxPartSlots];
#pragma unroll
        for (int s = 0; s < kMaxPartSlots; ++s)
            if (s < n_part) pv[s] = __ldcg(reinterpret_cast<const float4*>(part + (size_t)s * part_stride + (size_t)t * H) + c);
#pragma unroll
        for (int s = 0; s < kMaxPartSlots; ++s)
            if (s < n_part) { v.x += pv[s].x; v.y += pv[s].y; v.z += pv[s].z; v.w += pv[s].w; }
        reinterpret_cast<float4*>(srow)[c] = v;
        ss += v.x * v.x + v.y * v.y + v.z * v.z + v.w * v.w;
    }
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) ss += __shfl_xor_sync(0xffffffffu, ss, o);
    if ((threadIdx.x & 31) == 0) red[threadIdx.x >> 5] = ss;
    __syncthreads();
    float tot = 0.f;
#pragma unroll
    for (int w = 0; w < 8; ++w) tot += red[w];
    float rs = rsqrtf(tot / (float)H + eps);
    if (n_part > 0 || copy_from) {
        float4* out4 = reinterpret_cast<float4*>(resid + (size_t)t * H);
        for (int c = threadIdx.x; c < H / 4; c += blockDim.x) out4[c] = reinterpret_cast<float4*>(srow)[c];
    }
    if (xn != nullptr) {
        for (int c = threadIdx.x; c < H / 8; c += blockDim.x) {   // 8 consecutive features = one 16-byte group
            float4 a = reinterpret_cast<float4*>(srow)[2 * c], b = reinterpret_cast<float4*>(srow)[2 * c + 1];
            uint4 g = reinterpret_cast<const uint4*>(gain)[c];
            uint4 o;
            o.x = pack_bf16x2(__uint_as_float(g.x << 16) * (a.x * rs), __uint_as_float(g.x & 0xFFFF0000u) * (a.y * rs));
            o.y = pack_bf16x2(__uint_as_float(g.y << 16) * (a.z * rs), __uint_as_float(g.y & 0xFFFF0000u) * (a.w * rs));
            o.z = pack_bf16x2(__uint_as_float(g.z << 16) * (b.x * rs), __uint_as_float(g.z & 0xFFFF0000u) * (b.y * rs));
            o.w = pack_bf16x2(__uint_as_float(g.w << 16) * (b.z * rs), __uint_as_float(g.w & 0xFFFF0000u) * (b.w * rs));
            *reinterpret_cast<uint4*>(xn + packed_act_offset(t, c, n_pad)) = o;
        }
    }
}

// ---------------------------------------------------------------------------------------------
// Node list of a partial-tree forward: must be strictly ascending indices into a tree of T nodes.
// The layer's kernels index cache rows, mask rows and positions with it, so they are given a copy
// clamped into [0, T) (a malformed list then cannot reach outside the caller's buffers); the
// malformed list itself is reported through the status word.
// ---------------------------------------------------------------------------------------------
__global__ void __launch_bounds__(128) k_check_nodes(const int32_t* __restrict__ nodes, int m, int T, int32_t* __restrict__ clamped,
                                                     int32_t* __restrict__ d_status) {
    pdl_launch_dependents();
    pdl_wait();
    int j = threadIdx.x;
    if (j >= m) return;
    int n = nodes[j];
    bool bad = n < 0 || n >= T || (j > 0 && nodes[j - 1] >= n);
    clamped[j] = min(max(n, 0), T - 1);
    if (bad) report(d_status, CATS_ERR_INVALID_ARG);
}

// ---------------------------------------------------------------------------------------------
// Argmax over vocabulary tiles: the LM-head GEMM leaves, per 128-row vocabulary tile and node, the
// tile's maximum and the lowest index attaining it; one warp per node picks the overall winner
// (lowest index among equal maxima).
// ---------------------------------------------------------------------------------------------
// vmax (optional) receives the maximum itself, idx_offset is added to the winning index (a vocabulary shard reports global
// indices); the same kernel merges the shards' results, one "tile" per shard.
__global__ void __launch_bounds__(128) k_argmax_reduce(const float* __restrict__ pmax, const int32_t* __restrict__ pidx,
                                                       int n_tiles, int t_stride, int T, int32_t* __restrict__ amax,
                                                       float* __restrict__ vmax, int idx_offset) {
    pdl_launch_dependents();
    pdl_wait();
    int t = blockIdx.x * 4 + (threadIdx.x >> 5);
    int lane = threadIdx.x & 31;
    if (t >= T) return;
    float best = -INFINITY;
    int bi = 0x7fffffff;
    for (int k = lane; k < n_tiles; k += 32) {
        float v = pmax[(size_t)k * t_stride + t];
        int ix = pidx[(size_t)k * t_stride + t];
        if (v > best || (v == best && ix < bi)) { best = v; bi = ix; }
    }
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) {
        float ov = __shfl_xor_sync(0xffffffffu, best, o);
        int oi = __shfl_xor_sync(0xffffffffu, bi, o);
        if (ov > best || (ov == best && oi < bi)) { best = ov; bi = oi; }
    }
    if (lane == 0) {
        amax[t] = bi + idx_offset;
        if (vmax != nullptr) vmax[t] = best;
    }
}

// out[i] = part[0][i] + part[1][i] + ... (slot order): the split-K partial sums of a projection as ONE [T][hidden] fp32
// tensor, for a caller that reduces it across GPUs before the next norm folds it into the residual stream.
__global__ void __launch_bounds__(256) k_sum_parts(const float4* __restrict__ part, int n_part, size_t stride4, size_t n4,
                                                   float4* __restrict__ out) {
    pdl_launch_dependents();
    pdl_wait();
    for (size_t i = (size_t)blockIdx.x * blockDim.x + threadIdx.x; i < n4; i += (size_t)gridDim.x * blockDim.x) {
        float4 a = __ldcg(part + i);
        for (int s = 1; s < n_part; ++s) {
            const float4 q = __ldcg(part + (size_t)s * stride4 + i);
            a.x += q.x; a.y += q.y; a.z += q.z; a.w += q.w;
        }
        out[i] = a;
    }
}

// ---------------------------------------------------------------------------------------------
// The same reduction with the softmax statistics typical acceptance needs.  Tile k of node t carries
// its maximum m_k, Z_k = sum exp((l - m_k)/t) and S_k = sum exp((l - m_k)/t) (l - m_k).  With
// M = max_k m_k and w_k = exp((m_k - M)/t):
//   Z = sum_k w_k Z_k,   S = sum_k w_k (S_k + (m_k - M) Z_k)          (= sum_v e_v (l_v - M))
//   lse = M/t + log Z,   entropy = log Z - S / (t Z).
// Lanes take tiles in strides of 32 and the partial sums meet in a fixed shuffle order, so the
// result does not depend on timing.
// ---------------------------------------------------------------------------------------------
__global__ void __launch_bounds__(128) k_head_reduce(const float* __restrict__ pmax, const int32_t* __restrict__ pidx,
                                                     const float* __restrict__ psum, const float* __restrict__ ps1,
                                                     int n_tiles, int t_stride, int T, float inv_t,
                                                     int32_t* __restrict__ amax, float* __restrict__ lse,
                                                     float* __restrict__ entropy) {
    pdl_launch_dependents();
    pdl_wait();
    int t = blockIdx.x * 4 + (threadIdx.x >> 5);
    int lane = threadIdx.x & 31;
    if (t >= T) return;
    float best = -INFINITY;
    int bi = 0x7fffffff;
    for (int k = lane; k < n_tiles; k += 32) {
        float v = pmax[(size_t)k * t_stride + t];
        int ix = pidx[(size_t)k * t_stride + t];
        if (v > best || (v == best && ix < bi)) { best = v; bi = ix; }
    }
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) {
        float ov = __shfl_xor_sync(0xffffffffu, best, o);
        int oi = __shfl_xor_sync(0xffffffffu, bi, o);
        if (ov > best || (ov == best && oi < bi)) { best = ov; bi = oi; }
    }
    const float M = best;
    float Z = 0.f, S = 0.f;
    for (int k = lane; k < n_tiles; k += 32) {
        float d = pmax[(size_t)k * t_stride + t] - M;
        float w = exp2f(d * inv_t * 1.4426950408889634f);
        float zk = psum[(size_t)k * t_stride + t];
        Z = fmaf(w, zk, Z);
        S = fmaf(w, fmaf(d, zk, ps1[(size_t)k * t_stride + t]), S);
    }
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) {
        Z += __shfl_xor_sync(0xffffffffu, Z, o);
        S += __shfl_xor_sync(0xffffffffu, S, o);
    }
    if (lane == 0) {
        amax[t] = bi;
        float lz = logf(Z);
        lse[t] = fmaf(M, inv_t, lz);
        entropy[t] = lz - S * inv_t / Z;
    }
}

// ---------------------------------------------------------------------------------------------
// Greedy longest-accepted-path walk, one warp.  At node cur the target wants token argmax[cur];
// each lane tests four nodes, a ballot plus find-first-set gives the lowest matching child.
// ---------------------------------------------------------------------------------------------
__global__ void __launch_bounds__(32) k_walk(const int32_t* __restrict__ parent, const int32_t* __restrict__ tokens,
                                             const int32_t* __restrict__ amax, int T, int32_t* __restrict__ path,
                                             int32_t* __restrict__ path_len, int32_t* __restrict__ out_tokens,
                                             int32_t* __restrict__ n_out, int32_t* d_status) {
    pdl_launch_dependents();
    pdl_wait();
    int lane = threadIdx.x;
    int par[4], tok[4];
    bool bad = false;
#pragma unroll
    for (int q = 0; q < 4; ++q) {
        int j = q * 32 + lane;
        par[q] = j < T ? parent[j] : -2;
        tok[q] = j < T ? tokens[j] : -1;
        // Only an edge parent[j] < j can be followed, so the path is strictly increasing and never
        // longer than T whatever the array holds; a malformed entry is reported and leads nowhere.
        if (j < T && (j == 0 ? par[q] != -1 : (par[q] < 0 || par[q] >= j))) { bad = true; par[q] = -2; }
    }
    if (__any_sync(0xffffffffu, bad) && lane == 0) report(d_status, CATS_ERR_BAD_TREE);
    int cur = 0, len = 1, no = 0;
    if (lane == 0) path[0] = 0;
    for (int step = 0; step + 1 < T; ++step) {   // a path has at most T nodes
        int want = amax[cur];
        int next = -1;
#pragma unroll
        for (int q = 0; q < 4; ++q) {
            unsigned b = __ballot_sync(0xffffffffu, par[q] == cur && tok[q] == want);
            if (next < 0 && b) next = q * 32 + __ffs(b) - 1;
        }
        if (next < 0) break;
        if (lane == 0) { out_tokens[no] = want; path[len] = next; }
        ++no; ++len;
        cur = next;
    }
    if (lane == 0) {
        out_tokens[no] = amax[cur];
        *path_len = len;
        *n_out = no + 1;
    }
}

// ---------------------------------------------------------------------------------------------
// The walk under typical acceptance (Algorithm 1's loop with Acc = the relaxed criterion): child
// i of the current node is acceptable iff p_parent(token_i) > min(eps, delta * exp(-H_parent)),
// taken in the log domain with one fused multiply-add and one subtraction, both fp32 round to
// nearest:  fma(cand[i], 1/t, -lse[parent]) > min(log eps, log delta - entropy[parent]).
// The first acceptable child in node order is taken; the bonus token is the argmax at the last
// accepted node.
// ---------------------------------------------------------------------------------------------
__global__ void __launch_bounds__(32) k_walk_typical(const int32_t* __restrict__ parent, const int32_t* __restrict__ tokens,
                                                     const int32_t* __restrict__ amax, const float* __restrict__ cand,
                                                     const float* __restrict__ lse, const float* __restrict__ entropy, int T,
                                                     float inv_t, float log_eps, float log_delta, int32_t* __restrict__ path,
                                                     int32_t* __restrict__ path_len, int32_t* __restrict__ out_tokens,
                                                     int32_t* __restrict__ n_out) {
    pdl_launch_dependents();
    pdl_wait();
    int lane = threadIdx.x;
    int par[4], tok[4];
    bool ok[4];
#pragma unroll
    for (int q = 0; q < 4; ++q) {
        int j = q * 32 + lane;
        par[q] = j < T ? parent[j] : -2;
        tok[q] = j < T ? tokens[j] : -1;
        ok[q] = false;
        if (j > 0 && j < T && par[q] >= 0 && par[q] < j) {
            float logp = __fmaf_rn(cand[j], inv_t, -lse[par[q]]);
            float thr = fminf(log_eps, __fsub_rn(log_delta, entropy[par[q]]));
            ok[q] = logp > thr;
        }
    }
    int cur = 0, len = 1, no = 0;
    if (lane == 0) path[0] = 0;
    for (int step = 0; step < T; ++step) {
        int next = -1;
#pragma unroll
        for (int q = 0; q < 4; ++q) {
            unsigned b = __ballot_sync(0xffffffffu, par[q] == cur && ok[q]);
            if (next < 0 && b) next = q * 32 + __ffs(b) - 1;
        }
        if (next < 0) break;
        int t = 0;
#pragma unroll
        for (int q = 0; q < 4; ++q) {
            int v = __shfl_sync(0xffffffffu, tok[q], next & 31);
            if (q == (next >> 5)) t = v;
        }
        if (lane == 0) { out_tokens[no] = t; path[len] = next; }
        ++no; ++len;
        cur = next;
    }
    if (lane == 0) {
        out_tokens[no] = amax[cur];
        *path_len = len;
        *n_out = no + 1;
    }
}

// ---------------------------------------------------------------------------------------------
// KV compaction.  Each thread owns one 16-byte column slice of one cache (layer, K or V) and moves
// it for k = 0, 1, ... in order: row prefix+path[k] -> row prefix+k.  path[k] >= k and path is
// increasing, so a slice never reads a row it has already overwritten, and slices do not interact.
// ---------------------------------------------------------------------------------------------
__global__ void __launch_bounds__(256) k_compact(uint16_t* __restrict__ kc, uint16_t* __restrict__ vc, int n_layers,
                                                 long long layer_stride, long long row_elems, int prefix_len,
                                                 const int32_t* __restrict__ path, const int32_t* __restrict__ path_len,
                                                 int32_t* __restrict__ new_len, int32_t* __restrict__ src_rows,
                                                 int32_t* __restrict__ dst_rows, int32_t* d_status) {
    __shared__ int32_t sp[kMaxTree];
    __shared__ int bad;
    pdl_launch_dependents();
    pdl_wait();
    int n = *path_len;
    if (threadIdx.x == 0) bad = 0;
    __syncthreads();
    if (n < 1 || n > kMaxTree) {
        if (threadIdx.x == 0 && blockIdx.x == 0) report(d_status, CATS_ERR_INVALID_ARG);
        return;
    }
    for (int k = threadIdx.x; k < n; k += blockDim.x) {
        int p = path[k];
        sp[k] = p;
        if (p < k || p >= kMaxTree || (k > 0 && p <= path[k - 1])) bad = 1;
    }
    __syncthreads();
    if (bad) {
        if (threadIdx.x == 0 && blockIdx.x == 0) report(d_status, CATS_ERR_INVALID_ARG);
        return;
    }
    if (blockIdx.x == 0) {
        if (threadIdx.x == 0 && new_len) *new_len = prefix_len + n;
        for (int k = threadIdx.x; k < n; k += blockDim.x) {
            if (src_rows) src_rows[k] = prefix_len + sp[k];
            if (dst_rows) dst_rows[k] = prefix_len + k;
        }
    }
    long long slices_per_row = row_elems / 8;
    long long total = 2ll * n_layers * slices_per_row;
    for (long long s = (long long)blockIdx.x * blockDim.x + threadIdx.x; s < total; s += (long long)gridDim.x * blockDim.x) {
        long long col = s % slices_per_row;
        long long lw = s / slices_per_row;
        int layer = (int)(lw >> 1);
        uint16_t* base = ((lw & 1) ? vc : kc) + (size_t)layer * layer_stride + (size_t)col * 8;
        for (int k = 0; k < n; ++k) {
            int p = sp[k];
            if (p == k) continue;
            uint4 v = *reinterpret_cast<const uint4*>(base + (size_t)(prefix_len + p) * row_elems);
            *reinterpret_cast<uint4*>(base + (size_t)(prefix_len + k) * row_elems) = v;
        }
    }
}

// ---------------------------------------------------------------------------------------------
// launchers
// ---------------------------------------------------------------------------------------------
cudaError_t set_wait_limit_small(unsigned long long ns) { return cudaMemcpyToSymbol(g_wait_limit_ns, &ns, sizeof(ns)); }

// The same operation with the row held in registers and no dynamic shared memory, one row per CLUSTER of cs CTAs
// (cs = 1, 2 or 4): CTA `rank` owns columns [rank, rank + 1) * H / cs, NC float4 per thread, so that all loads of a
// thread are in flight at once; the sums of squares meet through distributed shared memory, added in rank order.
// Footprint: a CTA of this kernel fits on an SM beside a resident CTA of the projection kernel, so the projection that
// follows can already be resident and stream its first weight stages while the norm runs.  Thread pairs (even, odd
// lane) hold the two halves of one 16-byte group of the packed output.
#ifdef CATS_TIMELINE
static __device__ unsigned long long g_tl_norm[256 * kTlCtas * kTlStamps];
static int g_tl_norm_next = 0;
#define NORM_TL(slot) CATS_TL(tl, slot)
#define NORM_TL_PARAM , unsigned long long* tl
#else
#define NORM_TL(slot) do { } while (0)
#define NORM_TL_PARAM
#endif
// time-line stamps of k_rmsnorm_reg: 0 CTA entered, 2 dependency resolved, 3 row and partial sums summed, 9 CTA leaves
template <int NC>
__global__ void __launch_bounds__(256) k_rmsnorm_reg(float* __restrict__ resid, const float* __restrict__ copy_from,
                                                     const float* __restrict__ part, int n_part, size_t part_stride,
                                                     const uint16_t* __restrict__ gain, int H, float eps,
                                                     uint8_t* __restrict__ xn, int n_pad, const int32_t* __restrict__ pos,
                                                     const int32_t* __restrict__ nodes, float2* __restrict__ rope, int hd,
                                                     float rope_base, int* zero_flags, int n_flags, int cs,
                                                     int32_t* d_status, const WarmReq warm NORM_TL_PARAM) {
    __shared__ float red[8];
    __shared__ __align__(8) uint64_t xbar;     // completes when the partial sums of squares of all cs CTAs have landed
    __shared__ float slots[4];                 // slots[r]: the partial sum of the cluster's CTA r
    __shared__ int wait_expired;
    if (threadIdx.x == 0) NORM_TL(0);
    pdl_launch_dependents();
    const int t = blockIdx.x / cs, rank = blockIdx.x - t * cs;
    const int cols_cta = H / 4 / cs;          // float4 columns of this CTA
    const int col0 = rank * cols_cta;
    // everything that does not depend on the previous kernel: the exchange barrier and the gains
    if (cs > 1) {
        if (threadIdx.x == 0) {
            wait_expired = 0;
            mbar_init(&xbar, 1);
            mbar_fence_init();
            mbar_expect_tx(&xbar, 4u * (uint32_t)cs);
        }
        asm volatile("barrier.cluster.arrive.release.aligned;\n\tbarrier.cluster.wait.acquire.aligned;" ::: "memory");
    }
    uint2 g[NC];
#pragma unroll
    for (int j = 0; j < NC; ++j) {
        const int cl = threadIdx.x + 256 * j;
        g[j] = make_uint2(0u, 0u);
        if (xn != nullptr && cl < cols_cta) g[j] = __ldg(reinterpret_cast<const uint2*>(gain) + col0 + cl);
    }
    pdl_wait();
    if (threadIdx.x == 0) NORM_TL(2);
    if (zero_flags != nullptr && blockIdx.x == 0)
        for (int i = threadIdx.x; i < n_flags; i += blockDim.x) zero_flags[i] = 0;
    const float4* r4 = reinterpret_cast<const float4*>((copy_from ? copy_from : resid) + (size_t)t * H);
    float4 a[NC];
    float4 pv[NC][kMaxPartSlots / 2];
    // all loads first: the row, then the partial sums of the previous projection (slots 0..3 of every column)
#pragma unroll
    for (int j = 0; j < NC; ++j) {
        const int cl = threadIdx.x + 256 * j;
        a[j] = make_float4(0.f, 0.f, 0.f, 0.f);
        if (cl < cols_cta) a[j] = r4[col0 + cl];
    }
#pragma unroll
    for (int j = 0; j < NC; ++j) {
        const int cl = threadIdx.x + 256 * j;
#pragma unroll
        for (int s = 0; s < kMaxPartSlots / 2; ++s)
            if (s < n_part && cl < cols_cta)
                pv[j][s] = __ldcg(reinterpret_cast<const float4*>(part + (size_t)s * part_stride + (size_t)t * H) + col0 + cl);
    }
    // weights of the projection that follows, beyond what its own first copies fetch: requested into L2 while HBM is idle
    // (one thread of every warp, a few requests each, while the loads above are in flight)
    if ((threadIdx.x & 31) == 0) l2_warm(warm, blockIdx.x * 8 + (threadIdx.x >> 5), gridDim.x * 8, 8);
    // the rotary table of this node (fp64 so that large positions lose no accuracy): computed while the loads are in flight
    if (rope != nullptr && rank == cs - 1) {
        int half = hd / 2;
        int p = pos[nodes != nullptr ? nodes[t] : t];
        for (int i = threadIdx.x; i < half; i += blockDim.x) {
            double inv_freq = pow((double)rope_base, -2.0 * (double)i / (double)hd);
            double s, c;
            sincos((double)p * inv_freq, &s, &c);
            rope[(size_t)t * half + i] = make_float2((float)c, (float)s);
        }
    }
    float ss = 0.f;
#pragma unroll
    for (int j = 0; j < NC; ++j) {
        const int cl = threadIdx.x + 256 * j;
        if (cl >= cols_cta) continue;
        float4 v = a[j];
#pragma unroll
        for (int s = 0; s < kMaxPartSlots / 2; ++s)
            if (s < n_part) { v.x += pv[j][s].x; v.y += pv[j][s].y; v.z += pv[j][s].z; v.w += pv[j][s].w; }
        for (int s = kMaxPartSlots / 2; s < n_part; ++s) {     // more than four slots: rare (small matrices), in order
            const float4 q = __ldcg(reinterpret_cast<const float4*>(part + (size_t)s * part_stride + (size_t)t * H) + col0 + cl);
            v.x += q.x; v.y += q.y; v.z += q.z; v.w += q.w;
        }
        ss += v.x * v.x + v.y * v.y + v.z * v.z + v.w * v.w;
        a[j] = v;
    }
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) ss += __shfl_xor_sync(0xffffffffu, ss, o);
    if ((threadIdx.x & 31) == 0) red[threadIdx.x >> 5] = ss;
    __syncthreads();
    if (threadIdx.x == 0) NORM_TL(3);
    float tot = 0.f;
#pragma unroll
    for (int w = 0; w < 8; ++w) tot += red[w];
    const bool write_resid = n_part > 0 || copy_from != nullptr;
    float4* out4 = reinterpret_cast<float4*>(resid + (size_t)t * H);
    if (write_resid) {      // the new residual does not depend on the other CTAs' sums
#pragma unroll
        for (int j = 0; j < NC; ++j) {
            const int cl = threadIdx.x + 256 * j;
            if (cl < cols_cta) out4[col0 + cl] = a[j];
        }
    }
    if (cs > 1) {
        // every CTA sends its partial sum to slot [rank] of every CTA of the cluster (itself included); the store
        // signals the receiver's barrier, so one one-way trip through distributed shared memory is all that is waited for
        if (threadIdx.x == 0) {
            for (int r = 0; r < cs; ++r) {
                uint32_t rslot, rbar;
                asm volatile("mapa.shared::cluster.u32 %0, %1, %2;" : "=r"(rslot) : "r"(smem_u32(&slots[rank])), "r"(r));
                asm volatile("mapa.shared::cluster.u32 %0, %1, %2;" : "=r"(rbar) : "r"(smem_u32(&xbar)), "r"(r));
                asm volatile("st.async.weak.shared::cluster.mbarrier::complete_tx::bytes.b32 [%0], %1, [%2];"
                             ::"r"(rslot), "r"(__float_as_uint(tot)), "r"(rbar) : "memory");
            }
        }
        if (!mbar_wait(&xbar, 0, &wait_expired)) {
            if (threadIdx.x == 0) report(d_status, CATS_ERR_TIMEOUT);
        }
        tot = 0.f;
        for (int r = 0; r < cs; ++r) tot += slots[r];    // rank order: every CTA of the cluster gets the same bits
    }
    const float rs = rsqrtf(tot / (float)H + eps);
#pragma unroll
    for (int j = 0; j < NC; ++j) {
        const int cl = threadIdx.x + 256 * j;
        if (cl >= cols_cta) continue;
        const int c = col0 + cl;
        const float4 x = a[j];
        if (xn != nullptr) {
            uint2 o;
            o.x = pack_bf16x2(__uint_as_float(g[j].x << 16) * (x.x * rs), __uint_as_float(g[j].x & 0xFFFF0000u) * (x.y * rs));
            o.y = pack_bf16x2(__uint_as_float(g[j].y << 16) * (x.z * rs), __uint_as_float(g[j].y & 0xFFFF0000u) * (x.w * rs));
            *reinterpret_cast<uint2*>(xn + packed_act_offset(t, c >> 1, n_pad) + (size_t)(c & 1) * 8) = o;
        }
    }
    if (threadIdx.x == 0) NORM_TL(9);
}

template <typename Kern, typename... Args>
static cudaError_t launch_cluster_pdl(Kern kernel, dim3 grid, dim3 block, int cs, cudaStream_t st, Args... args) {
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = grid;
    cfg.blockDim = block;
    cfg.dynamicSmemBytes = 0;
    cfg.stream = st;
    cudaLaunchAttribute attr[2];
    int n = 0;
    if (cs > 1) {
        attr[n].id = cudaLaunchAttributeClusterDimension;
        attr[n].val.clusterDim.x = (unsigned)cs;
        attr[n].val.clusterDim.y = 1;
        attr[n].val.clusterDim.z = 1;
        ++n;
    }
    if (!g_call_boundary) {
        attr[n].id = cudaLaunchAttributeProgrammaticStreamSerialization;
        attr[n].val.programmaticStreamSerializationAllowed = 1;
        ++n;
    }
    g_call_boundary = false;
    cfg.attrs = attr;
    cfg.numAttrs = n;
    ++g_launch_count;
    return cudaLaunchKernelEx(&cfg, kernel, args...);
}

cudaError_t launch_mask_pos(const int32_t* parent, int T, int prefix_len, uint64_t* mask, int32_t* pos, int32_t* depth,
                            int32_t* d_status, cudaStream_t st) {
    return launch_pdl(k_mask_pos, dim3(1), dim3(kMaxTree), 0, st, parent, T, prefix_len, mask, pos, depth, d_status);
}

cudaError_t launch_embed(const void* E, const int32_t* tokens, int T, int H, int vocab, float* resid, int32_t* d_status,
                         cudaStream_t st) {
    return launch_pdl(k_embed, dim3(T), dim3(256), 0, st, (const uint16_t*)E, tokens, H, vocab, resid, d_status);
}

cudaError_t launch_rmsnorm(float* resid, const float* copy_from, const float* part, int n_part, size_t part_stride,
                           const void* gain, int T, int H, float eps, void* xn_packed, const int32_t* pos, const int32_t* nodes,
                           float2* rope, int hd, float rope_base, int* zero_flags, int n_flags, cudaStream_t st,
                           int32_t* d_status, const WarmReq* warm_in) {
    const int n_pad = (T + 15) / 16 * 16;
#ifdef CATS_TIMELINE
    unsigned long long* tl_ptr = nullptr;
    cudaGetSymbolAddress((void**)&tl_ptr, g_tl_norm);
    tl_ptr += (size_t)(g_tl_norm_next++ % 256) * kTlCtas * kTlStamps;
#define NORM_TL_ARG , tl_ptr
#else
#define NORM_TL_ARG
#endif
    const WarmReq warm = warm_in ? warm_req(warm_in->ptr, warm_in->bytes, warm_in->period, warm_in->phase) : warm_req(nullptr, 0, 0, 0);
#define CATS_NORM_REG(NC)                                                                                                   \
    return launch_cluster_pdl(k_rmsnorm_reg<NC>, dim3(T * cs), dim3(256), cs, st, resid, copy_from, part, n_part, part_stride, \
                              (const uint16_t*)gain, H, eps, (uint8_t*)xn_packed, n_pad, pos, nodes, rope, hd, rope_base,    \
                              zero_flags, n_flags, cs, d_status, warm NORM_TL_ARG)
#ifndef CATS_NORM_SMEM
    {
        // as many CTAs per row as keep the grid within one wave and leave every CTA at least 256 columns
        const int n_cols = H / 4;
        int cs = 1;
        for (int c = 4; c >= 2; c >>= 1)
            if (T * c <= 148 && n_cols % c == 0 && n_cols / c >= 256) { cs = c; break; }
        const int nc = (n_cols / cs + 255) / 256;
        if (nc <= 1) CATS_NORM_REG(1);
        if (nc <= 2) CATS_NORM_REG(2);
        if (nc <= 4) CATS_NORM_REG(4);
        if (nc <= 5) CATS_NORM_REG(5);
        if (nc <= 8) CATS_NORM_REG(8);
    }
#endif
#undef CATS_NORM_REG
    return launch_pdl(k_rmsnorm, dim3(T), dim3(256), (size_t)H * sizeof(float), st, resid, copy_from, part, n_part,
                      part_stride, (const uint16_t*)gain, H, eps, (uint8_t*)xn_packed, n_pad, pos, nodes, rope,
                      hd, rope_base, zero_flags, n_flags);
}

// Time line of the k_rmsnorm_reg launches (measurement builds): copies the stamps to the host, or clears them.
cudaError_t timeline_norm(void* host, size_t bytes, bool clear) {
#ifdef CATS_TIMELINE
    if (clear) {
        void* b = nullptr;
        cudaError_t e = cudaGetSymbolAddress(&b, g_tl_norm);
        g_tl_norm_next = 0;
        return e != cudaSuccess ? e : cudaMemset(b, 0, sizeof(g_tl_norm));
    }
    return cudaMemcpyFromSymbol(host, g_tl_norm, bytes < sizeof(g_tl_norm) ? bytes : sizeof(g_tl_norm));
#else
    (void)host; (void)bytes; (void)clear;
    return cudaErrorNotSupported;
#endif
}

cudaError_t launch_check_nodes(const int32_t* nodes, int m, int T, int32_t* clamped, int32_t* d_status, cudaStream_t st) {
    return launch_pdl(k_check_nodes, dim3(1), dim3(128), 0, st, nodes, m, T, clamped, d_status);
}

cudaError_t launch_argmax_reduce(const float* pmax, const int32_t* pidx, int n_tiles, int t_stride, int T, int32_t* amax,
                                 float* vmax, int idx_offset, cudaStream_t st) {
    return launch_pdl(k_argmax_reduce, dim3((T + 3) / 4), dim3(128), 0, st, pmax, pidx, n_tiles, t_stride, T, amax, vmax, idx_offset);
}

cudaError_t launch_sum_parts(const float* part, int n_part, size_t part_stride, size_t n, float* out, cudaStream_t st) {
    const size_t n4 = n / 4;
    int blocks = (int)((n4 + 255) / 256);
    if (blocks > 148 * 4) blocks = 148 * 4;
    if (blocks < 1) blocks = 1;
    return launch_pdl(k_sum_parts, dim3(blocks), dim3(256), 0, st, (const float4*)part, n_part, part_stride / 4, n4, (float4*)out);
}

cudaError_t launch_head_reduce(const float* pmax, const int32_t* pidx, const float* psum, const float* ps1, int n_tiles,
                               int t_stride, int T, float inv_temperature, int32_t* amax, float* lse, float* entropy,
                               cudaStream_t st) {
    return launch_pdl(k_head_reduce, dim3((T + 3) / 4), dim3(128), 0, st, pmax, pidx, psum, ps1, n_tiles, t_stride, T,
                      inv_temperature, amax, lse, entropy);
}

cudaError_t launch_walk_typical(const int32_t* parent, const int32_t* tokens, const int32_t* amax, const float* cand,
                                const float* lse, const float* entropy, int T, float inv_temperature, float log_eps,
                                float log_delta, int32_t* path, int32_t* path_len, int32_t* out_tokens, int32_t* n_out,
                                cudaStream_t st) {
    return launch_pdl(k_walk_typical, dim3(1), dim3(32), 0, st, parent, tokens, amax, cand, lse, entropy, T, inv_temperature,
                      log_eps, log_delta, path, path_len, out_tokens, n_out);
}

cudaError_t launch_walk(const int32_t* parent, const int32_t* tokens, const int32_t* amax, int T, int32_t* path,
                        int32_t* path_len, int32_t* out_tokens, int32_t* n_out, int32_t* d_status, cudaStream_t st) {
    return launch_pdl(k_walk, dim3(1), dim3(32), 0, st, parent, tokens, amax, T, path, path_len, out_tokens, n_out, d_status);
}

cudaError_t launch_compact(void* kc, void* vc, int n_layers, long long layer_stride, long long row_elems, int prefix_len,
                           const int32_t* path, const int32_t* path_len, int32_t* new_len, int32_t* src_rows,
                           int32_t* dst_rows, int32_t* d_status, cudaStream_t st) {
    long long total = 2ll * n_layers * (row_elems / 8);
    int blocks = (int)((total + 255) / 256);
    if (blocks > 148 * 8) blocks = 148 * 8;
    if (blocks < 1) blocks = 1;
    return launch_pdl(k_compact, dim3(blocks), dim3(256), 0, st, (uint16_t*)kc, (uint16_t*)vc, n_layers, layer_stride,
                      row_elems, prefix_len, path, path_len, new_len, src_rows, dst_rows, d_status);
}

}  // namespace cats
