// Tree-masked attention of the T draft-tree nodes against the KV prefix plus their own ancestors.
//
// Two kernels: k_tree_attn (bf16 mma.sync; head_dim 64 or 128), described first, and k_tree_attn_tc (tcgen05, tensor
// memory and TMA), further down, which takes every head_dim-128 problem.
//
// Q [T_pad][hd] sits in shared memory; the cache rows stream through a double-buffered cp.async pipeline
// (128-bit loads); S = Q K^T and O += P V run on bf16 tensor-core MMAs (fp32 accumulation, online softmax in
// fp32 with warp-shuffle row reductions, the probabilities as a bf16 pair hi + lo).  Prefix rows need no mask;
// rows >= prefix_len test bit (row - prefix) of the node's 128-bit ancestor mask held in shared memory.
// Warps are laid out as (16-row query tile) x (slice of the block of rows), so small trees still use every
// warp; every warp leaves its partial (m, l, O) in its CTA's shared memory.  Two ways of dividing a head:
//   * query split (trees of four or more query tiles over a short cache): the CTAs of a head take different
//     query tiles, every CTA reads all rows and merges its warps' partials alone;
//   * split-KV inside a thread-block cluster (up to 8 CTAs): the rows are divided among the CTAs; each CTA
//     pushes, per destination, the records of the query rows that destination merges, with bulk copies through
//     distributed shared memory completing on the destination's mbarrier; the merge reads local memory only.
// The merge is by log-sum-exp in a fixed order; the result is written as bf16.  Only when a head has far more
// rows than a cluster can cover with few heads (long prefixes, few heads) are several clusters used per head;
// their merged partials then go to the caller's workspace and k_attn_combine merges them.
#include <mutex>

#include "cats_kernels.cuh"

namespace cats {

constexpr int kAttnThreads = 256;
constexpr int kKvBlock = 64;

__device__ __forceinline__ void cp_async16(void* smem_dst, const void* gsrc) {
    asm volatile("cp.async.cg.shared.global [%0], [%1], 16;" ::"r"(smem_u32(smem_dst)), "l"(gsrc) : "memory");
}
__device__ __forceinline__ void cp_async_commit() { asm volatile("cp.async.commit_group;" ::: "memory"); }
template <int N>
__device__ __forceinline__ void cp_async_wait() { asm volatile("cp.async.wait_group %0;" ::"n"(N) : "memory"); }

__device__ __forceinline__ void ldmatrix_x4(uint32_t addr, uint32_t& r0, uint32_t& r1, uint32_t& r2, uint32_t& r3) {
    asm volatile("ldmatrix.sync.aligned.m8n8.x4.shared.b16 {%0,%1,%2,%3}, [%4];" : "=r"(r0), "=r"(r1), "=r"(r2), "=r"(r3) : "r"(addr));
}
__device__ __forceinline__ void ldmatrix_x4_trans(uint32_t addr, uint32_t& r0, uint32_t& r1, uint32_t& r2, uint32_t& r3) {
    asm volatile("ldmatrix.sync.aligned.m8n8.x4.trans.shared.b16 {%0,%1,%2,%3}, [%4];" : "=r"(r0), "=r"(r1), "=r"(r2), "=r"(r3) : "r"(addr));
}
__device__ __forceinline__ void mma_bf16_16816(float* c, const uint32_t* a, uint32_t b0, uint32_t b1) {
    asm volatile("mma.sync.aligned.m16n8k16.row.col.f32.bf16.bf16.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%0,%1,%2,%3};"
                 : "+f"(c[0]), "+f"(c[1]), "+f"(c[2]), "+f"(c[3])
                 : "r"(a[0]), "r"(a[1]), "r"(a[2]), "r"(a[3]), "r"(b0), "r"(b1));
}

// byte offset of 16-byte chunk `chunk` of row `row` in a [rows][HD] bf16 tile with XOR swizzle
template <int HD>
__device__ __forceinline__ uint32_t tile_off(int row, int chunk) {
    return (uint32_t)(row * (HD * 2) + ((chunk ^ (row & 7)) << 4));
}

struct AttnDev {
    const uint16_t *q, *k, *v;
    const uint64_t* mask;
    const int32_t* nodes;   // null, or the tree node of each query row (selects its mask row)
    int Tk;                 // tree rows in the cache after the prefix
    int rpr;                // query rows each CTA of a cluster merges (contiguous block)
    int qsplit;             // > 0: the CTAs of a head split the QUERY tiles (n_mt tiles each) and every CTA reads all rows
    int stages;             // tcgen05 kernel: stages of the K/V ring
    int32_t* d_status;
    int T, P, nh, n_mt, kvg, csize, n_outer, rows_per_split, blk, kv_area;   // blk: cache rows per pipeline block (multiple of 16*kvg); kv_area: bytes of the K/V buffers
    long long kv_stride;
    float scale_log2;
    int out_npad;        // > 0: out is in the packed activation layout with this many rows per K block
    uint16_t* out;
    float* part_o;       // n_outer > 1: [nh][n_outer][T_pad][hd] fp32
    float* part_ml;      //              [nh][n_outer][T_pad][2]
    int dbg_skip_q;      // fault injection (tcgen05 kernel): the loader announces Q but never copies it
    WarmReq warm[3];     // see AttnProblem
    int recv_over_ring;  // tcgen05 kernel: the records deposited by the cluster's CTAs lie over the K/V ring (see the kernel)
#ifdef CATS_TIMELINE
    unsigned long long* tl;      // this launch's time-line slot
#endif
};
#ifdef CATS_TIMELINE
#define ATTN_TL(slot) CATS_TL(p.tl, slot)
static __device__ unsigned long long g_tl_attn[128 * kTlCtas * kTlStamps];
static int g_tl_attn_next = 0;
#else
#define ATTN_TL(slot) do { } while (0)
#endif
// time-line stamps of the tcgen05 kernel: 0 CTA entered, 1 set-up done, 2 dependency resolved, 3 dependent copies issued,
// 4 Q and the first block landed, 5 first Q K^T issued, 6 first S complete, 7 last P written, 8 last P V complete,
// 9 records deposited, 10 records published (cluster barrier), 11 merged, CTA leaves

__device__ __forceinline__ void cluster_sync_all() {
    asm volatile("barrier.cluster.arrive.release.aligned;\n\tbarrier.cluster.wait.acquire.aligned;" ::: "memory");
}
__device__ __forceinline__ uint32_t cluster_map(uint32_t local_smem_addr, int rank) {
    uint32_t r;
    asm volatile("mapa.shared::cluster.u32 %0, %1, %2;" : "=r"(r) : "r"(local_smem_addr), "r"(rank));
    return r;
}
__device__ __forceinline__ float2 ld_cluster_f2(uint32_t addr) {
    float2 v;
    asm volatile("ld.shared::cluster.v2.f32 {%0,%1}, [%2];" : "=f"(v.x), "=f"(v.y) : "r"(addr) : "memory");
    return v;
}
__device__ __forceinline__ float4 ld_cluster_f4(uint32_t addr) {
    float4 v;
    asm volatile("ld.shared::cluster.v4.f32 {%0,%1,%2,%3}, [%4];" : "=f"(v.x), "=f"(v.y), "=f"(v.z), "=f"(v.w) : "r"(addr));
    return v;
}

template <int HD, bool K32>
__global__ void __launch_bounds__(kAttnThreads, 1) k_tree_attn(const AttnDev p) {
    extern __shared__ __align__(128) uint8_t sm[];
    constexpr int ROWB = HD * 2;                 // bytes per tile row
    constexpr int NCH = HD / 8;                  // 16-byte chunks per row
    constexpr int KS = HD / 16;                  // k-steps of Q K^T
    constexpr int NT = HD / 8;                   // n-tiles of the output
    uint8_t* q_s = sm;                                           // [n_mt*16][HD]
    uint8_t* kv_s = q_s + (size_t)p.n_mt * 16 * ROWB;            // 2 buffers x (K [64][HD], V [64][HD])
    uint64_t* mask_s = reinterpret_cast<uint64_t*>(kv_s + p.kv_area);   // [n_mt*16][2]
    float* recv = reinterpret_cast<float*>(mask_s + (size_t)p.n_mt * 16 * 2);   // [csize][kvg][rpr][HD + 4]: partials pushed by the cluster
    uint64_t* rbar = reinterpret_cast<uint64_t*>(recv + (size_t)p.csize * p.kvg * p.rpr * (HD + 4));
    volatile int* wait_expired = reinterpret_cast<volatile int*>(rbar + 1);

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int split = p.qsplit > 0 ? 0 : (int)blockIdx.x, h = blockIdx.y;
    const int row_base = p.qsplit > 0 ? (int)blockIdx.x * p.n_mt * 16 : 0;   // first query row of this CTA
    const int S = p.P + p.Tk;
    const int c_begin = min(S, split * p.rows_per_split);
    const int c_end = min(S, c_begin + p.rows_per_split);
    const int nb = (c_end - c_begin + p.blk - 1) / p.blk;
    const int mt = warp % p.n_mt, g = warp / p.n_mt;
    const bool active = g < p.kvg;
    const int R = p.blk / p.kvg;                 // rows of each block this warp's group handles
    const int Tpad = p.n_mt * 16;

    auto load_kv = [&](int b, int buf) {
        uint8_t* ks = kv_s + (size_t)buf * 2 * p.blk * ROWB;
        uint8_t* vs = ks + p.blk * ROWB;
        int r0 = c_begin + b * p.blk;
        for (int e = threadIdx.x; e < p.blk * NCH; e += kAttnThreads) {
            int r = e / NCH, ch = e % NCH;
            int row = r0 + r;
            uint32_t off = tile_off<HD>(r, ch);
            if (row < c_end) {
                size_t gofs = (size_t)row * p.kv_stride + (size_t)h * HD + ch * 8;
                cp_async16(ks + off, p.k + gofs);
                cp_async16(vs + off, p.v + gofs);
            } else {
                *reinterpret_cast<uint4*>(ks + off) = make_uint4(0, 0, 0, 0);
                *reinterpret_cast<uint4*>(vs + off) = make_uint4(0, 0, 0, 0);
            }
        }
    };

    pdl_launch_dependents();
    // the first block can be requested before the previous kernel has finished if it lies in the prefix
    const bool early = (c_begin + p.blk <= p.P);
    if (early) load_kv(0, 0);
    // with a second buffer and a second block inside the prefix, that one too
    const bool early2 = early && nb > 1 && p.kv_area >= 4 * p.blk * ROWB && c_begin + 2 * p.blk <= p.P;
    if (early2) load_kv(1, 1);
    if (p.csize > 1) {
        // the barrier the cluster's pushed partials complete on; visible to the peers before anybody can send
        if (threadIdx.x == 0) {
            const int rank_ = split % p.csize;
            const int r0 = min(Tpad, rank_ * p.rpr), r1 = min(Tpad, r0 + p.rpr);
            *wait_expired = 0;
            mbar_init(rbar, 1);
            mbar_fence_init();
            mbar_expect_tx(rbar, (uint32_t)(r1 - r0) * (HD + 4) * 4u * (uint32_t)(p.csize * p.kvg));
        }
        cluster_sync_all();
    }
    pdl_wait();
    for (int e = threadIdx.x; e < Tpad * NCH; e += kAttnThreads) {
        int r = e / NCH, ch = e % NCH;
        uint32_t off = tile_off<HD>(r, ch);
        if (row_base + r < p.T) cp_async16(q_s + off, p.q + ((size_t)(row_base + r) * p.nh + h) * HD + ch * 8);
        else *reinterpret_cast<uint4*>(q_s + off) = make_uint4(0, 0, 0, 0);
    }
    for (int e = threadIdx.x; e < Tpad * 2; e += kAttnThreads) {
        uint64_t w = 0ull;
        const int gr = row_base + (e >> 1);
        if (gr < p.T) w = p.mask[(size_t)(p.nodes != nullptr ? p.nodes[gr] : gr) * 2 + (e & 1)];
        mask_s[e] = w;
    }
    if (!early && nb > 0) load_kv(0, 0);
    cp_async_commit();

    uint32_t qf[KS][4];
    float o[NT][4];
#pragma unroll
    for (int j = 0; j < NT; ++j) { o[j][0] = o[j][1] = o[j][2] = o[j][3] = 0.f; }
    float m_run[2] = {-INFINITY, -INFINITY}, l_run[2] = {0.f, 0.f};
    const int row_a = mt * 16 + (lane >> 2), row_b = row_a + 8;   // the two query rows this thread owns

    for (int b = 0; b < nb; ++b) {
        if (b + 1 < nb) {
            if (!(b == 0 && early2)) load_kv(b + 1, (b + 1) & 1);
            cp_async_commit();
            cp_async_wait<1>();
        } else {
            cp_async_wait<0>();
        }
        __syncthreads();
        if (b == 0 && active) {
#pragma unroll
            for (int ks = 0; ks < KS; ++ks) {
                int r = mt * 16 + (lane & 15), ch = ks * 2 + (lane >> 4);
                ldmatrix_x4(smem_u32(q_s + tile_off<HD>(r, ch)), qf[ks][0], qf[ks][1], qf[ks][2], qf[ks][3]);
            }
        }
        if (active) {
            const uint8_t* ks_s = kv_s + (size_t)(b & 1) * 2 * p.blk * ROWB;
            const uint8_t* vs_s = ks_s + p.blk * ROWB;
            const int rbase = g * R;                              // first row of this warp's slice in the block
            const int cbase = c_begin + b * p.blk + rbase;     // its global cache row
            // 16 rows of the slice at a time: S = Q K^T (16 x 16), mask, online softmax, O += P V
            for (int sub = 0; sub < R; sub += 16) {
                if (cbase + sub >= c_end) break;
                if (K32 && sub + 32 <= R && cbase + sub + 32 <= min(p.P, c_end)) {
                    // 32 prefix rows at once (all visible): the softmax bookkeeping is paid once for twice the keys and
                    // the four score tiles are four independent chains of MMAs
                    float s[4][4];
#pragma unroll
                    for (int n = 0; n < 4; ++n) { s[n][0] = s[n][1] = s[n][2] = s[n][3] = 0.f; }
#pragma unroll
                    for (int ks = 0; ks < KS; ++ks) {
                        uint32_t b0, b1, b2, b3, c0, c1, c2, c3;
                        const int r = rbase + sub + (lane & 7) + ((lane >> 4) << 3), ch = ks * 2 + ((lane >> 3) & 1);
                        ldmatrix_x4(smem_u32(ks_s + tile_off<HD>(r, ch)), b0, b1, b2, b3);
                        ldmatrix_x4(smem_u32(ks_s + tile_off<HD>(r + 16, ch)), c0, c1, c2, c3);
                        mma_bf16_16816(s[0], qf[ks], b0, b1);
                        mma_bf16_16816(s[1], qf[ks], b2, b3);
                        mma_bf16_16816(s[2], qf[ks], c0, c1);
                        mma_bf16_16816(s[3], qf[ks], c2, c3);
                    }
                    float mx_a = -INFINITY, mx_b = -INFINITY;
#pragma unroll
                    for (int n = 0; n < 4; ++n) {
#pragma unroll
                        for (int e = 0; e < 4; ++e) s[n][e] *= p.scale_log2;
                        mx_a = fmaxf(mx_a, fmaxf(s[n][0], s[n][1]));
                        mx_b = fmaxf(mx_b, fmaxf(s[n][2], s[n][3]));
                    }
                    mx_a = fmaxf(mx_a, __shfl_xor_sync(0xffffffffu, mx_a, 1));
                    mx_a = fmaxf(mx_a, __shfl_xor_sync(0xffffffffu, mx_a, 2));
                    mx_b = fmaxf(mx_b, __shfl_xor_sync(0xffffffffu, mx_b, 1));
                    mx_b = fmaxf(mx_b, __shfl_xor_sync(0xffffffffu, mx_b, 2));
                    const float mn_a = fmaxf(m_run[0], mx_a), mn_b = fmaxf(m_run[1], mx_b);   // finite: prefix rows are visible
                    const float corr_a = exp2f(m_run[0] - mn_a), corr_b = exp2f(m_run[1] - mn_b);
                    m_run[0] = mn_a; m_run[1] = mn_b;
                    float la = 0.f, lb = 0.f;
#pragma unroll
                    for (int n = 0; n < 4; ++n) {
                        s[n][0] = exp2f(s[n][0] - mn_a); s[n][1] = exp2f(s[n][1] - mn_a);
                        s[n][2] = exp2f(s[n][2] - mn_b); s[n][3] = exp2f(s[n][3] - mn_b);
                        la += s[n][0] + s[n][1];
                        lb += s[n][2] + s[n][3];
                    }
                    l_run[0] = l_run[0] * corr_a + la;
                    l_run[1] = l_run[1] * corr_b + lb;
                    if (__any_sync(0xffffffffu, corr_a != 1.f || corr_b != 1.f)) {
#pragma unroll
                        for (int j = 0; j < NT; ++j) { o[j][0] *= corr_a; o[j][1] *= corr_a; o[j][2] *= corr_b; o[j][3] *= corr_b; }
                    }
#pragma unroll
                    for (int kk = 0; kk < 2; ++kk) {            // the two 16-key halves of the P V product
                        uint32_t pa[4], pl[4];
#pragma unroll
                        for (int e = 0; e < 4; ++e) {
                            const float x0 = s[2 * kk + (e >> 1)][(e & 1) * 2], x1 = s[2 * kk + (e >> 1)][(e & 1) * 2 + 1];
                            const float h0 = bf16_bits_to_float(float_to_bf16_bits(x0));
                            const float h1 = bf16_bits_to_float(float_to_bf16_bits(x1));
                            pa[e] = pack_bf16x2(h0, h1);
                            pl[e] = pack_bf16x2(x0 - h0, x1 - h1);
                        }
#pragma unroll
                        for (int j = 0; j < NT; j += 2) {
                            uint32_t b0, b1, b2, b3;
                            const int r = rbase + sub + kk * 16 + (lane & 15), ch = j + (lane >> 4);
                            ldmatrix_x4_trans(smem_u32(vs_s + tile_off<HD>(r, ch)), b0, b1, b2, b3);
                            mma_bf16_16816(o[j], pa, b0, b1);
                            mma_bf16_16816(o[j], pl, b0, b1);
                            mma_bf16_16816(o[j + 1], pa, b2, b3);
                            mma_bf16_16816(o[j + 1], pl, b2, b3);
                        }
                    }
                    sub += 16;      // the loop adds the other 16
                    continue;
                }
                // two accumulator pairs (even and odd k-steps): the chain of dependent MMAs is half as long
                float s0[4] = {0.f, 0.f, 0.f, 0.f}, s1[4] = {0.f, 0.f, 0.f, 0.f};
                float t0[4] = {0.f, 0.f, 0.f, 0.f}, t1[4] = {0.f, 0.f, 0.f, 0.f};
#pragma unroll
                for (int ks = 0; ks < KS; ks += 2) {
                    uint32_t b0, b1, b2, b3, c0, c1, c2, c3;
                    const int r = rbase + sub + (lane & 7) + ((lane >> 4) << 3), ch = ks * 2 + ((lane >> 3) & 1);
                    ldmatrix_x4(smem_u32(ks_s + tile_off<HD>(r, ch)), b0, b1, b2, b3);
                    ldmatrix_x4(smem_u32(ks_s + tile_off<HD>(r, ch + 2)), c0, c1, c2, c3);
                    mma_bf16_16816(s0, qf[ks], b0, b1);
                    mma_bf16_16816(s1, qf[ks], b2, b3);
                    mma_bf16_16816(t0, qf[ks + 1], c0, c1);
                    mma_bf16_16816(t1, qf[ks + 1], c2, c3);
                }
#pragma unroll
                for (int e = 0; e < 4; ++e) { s0[e] += t0[e]; s1[e] += t1[e]; }
                // visibility of the 4+4 scores this thread holds
                float sc[8];
                if (cbase + sub + 16 <= p.P) {
                    // 16 prefix rows: every one visible to every node
#pragma unroll
                    for (int e = 0; e < 8; ++e) sc[e] = ((e >> 2) ? s1[e & 3] : s0[e & 3]) * p.scale_log2;
                } else {
                    const uint64_t ma0 = mask_s[row_a * 2], ma1 = mask_s[row_a * 2 + 1];
                    const uint64_t mb0 = mask_s[row_b * 2], mb1 = mask_s[row_b * 2 + 1];
#pragma unroll
                    for (int e = 0; e < 8; ++e) {
                        int nt = e >> 2, ee = e & 3;
                        int col = cbase + sub + nt * 8 + (lane & 3) * 2 + (ee & 1);
                        bool rowb = (ee >> 1) != 0;
                        bool vis;
                        if (col < p.P) vis = true;
                        else if (col >= S) vis = false;
                        else {
                            int j = col - p.P;
                            uint64_t w = rowb ? (j < 64 ? mb0 : mb1) : (j < 64 ? ma0 : ma1);
                            vis = (w >> (j & 63)) & 1ull;
                        }
                        float v = (nt ? s1[ee] : s0[ee]) * p.scale_log2;
                        sc[e] = vis ? v : -INFINITY;
                    }
                }
                float mx_a = fmaxf(fmaxf(sc[0], sc[1]), fmaxf(sc[4], sc[5]));
                float mx_b = fmaxf(fmaxf(sc[2], sc[3]), fmaxf(sc[6], sc[7]));
                mx_a = fmaxf(mx_a, __shfl_xor_sync(0xffffffffu, mx_a, 1));
                mx_a = fmaxf(mx_a, __shfl_xor_sync(0xffffffffu, mx_a, 2));
                mx_b = fmaxf(mx_b, __shfl_xor_sync(0xffffffffu, mx_b, 1));
                mx_b = fmaxf(mx_b, __shfl_xor_sync(0xffffffffu, mx_b, 2));
                float mn_a = fmaxf(m_run[0], mx_a), mn_b = fmaxf(m_run[1], mx_b);
                float ref_a = (mn_a == -INFINITY) ? 0.f : mn_a, ref_b = (mn_b == -INFINITY) ? 0.f : mn_b;
                float corr_a = exp2f(m_run[0] - ref_a), corr_b = exp2f(m_run[1] - ref_b);
                m_run[0] = mn_a; m_run[1] = mn_b;
                float pr[8];
#pragma unroll
                for (int e = 0; e < 8; ++e) pr[e] = exp2f(sc[e] - (((e & 3) >> 1) ? ref_b : ref_a));
                l_run[0] = l_run[0] * corr_a + pr[0] + pr[1] + pr[4] + pr[5];
                l_run[1] = l_run[1] * corr_b + pr[2] + pr[3] + pr[6] + pr[7];
                if (__any_sync(0xffffffffu, corr_a != 1.f || corr_b != 1.f)) {   // a running maximum moved: rescale O
#pragma unroll
                    for (int j = 0; j < NT; ++j) { o[j][0] *= corr_a; o[j][1] *= corr_a; o[j][2] *= corr_b; o[j][3] *= corr_b; }
                }
                // The probabilities enter the P V product as bf16 pairs hi + lo (hi = bf16(p), lo = bf16(p - hi)),
                // so the product carries ~16 mantissa bits of p instead of 8; V is bf16 exactly.
                uint32_t pa[4], pl[4];
#pragma unroll
                for (int e = 0; e < 4; ++e) {
                    float h0 = bf16_bits_to_float(float_to_bf16_bits(pr[2 * e]));
                    float h1 = bf16_bits_to_float(float_to_bf16_bits(pr[2 * e + 1]));
                    pa[e] = pack_bf16x2(h0, h1);
                    pl[e] = pack_bf16x2(pr[2 * e] - h0, pr[2 * e + 1] - h1);
                }
#pragma unroll
                for (int j = 0; j < NT; j += 2) {
                    uint32_t b0, b1, b2, b3;
                    int r = rbase + sub + (lane & 15), ch = j + (lane >> 4);
                    ldmatrix_x4_trans(smem_u32(vs_s + tile_off<HD>(r, ch)), b0, b1, b2, b3);
                    mma_bf16_16816(o[j], pa, b0, b1);
                    mma_bf16_16816(o[j], pl, b0, b1);
                    mma_bf16_16816(o[j + 1], pa, b2, b3);
                    mma_bf16_16816(o[j + 1], pl, b2, b3);
                }
            }
        }
        __syncthreads();
    }

    // ---- every warp deposits its partial (m, l, O); the cluster merges all partials of the head ----
    // Record of one (partial, query row): HD floats of O, then m, l and two pad floats (a multiple of 16 bytes).
    // The query rows are divided among the CTAs of the cluster in contiguous blocks of rpr rows; every CTA PUSHES, for
    // every destination CTA, the slab of records that CTA will merge, with bulk copies through distributed shared
    // memory that complete on the destination's mbarrier.  The merge then reads local shared memory only.
    constexpr int REC = HD + 4;
    l_run[0] += __shfl_xor_sync(0xffffffffu, l_run[0], 1);
    l_run[0] += __shfl_xor_sync(0xffffffffu, l_run[0], 2);
    l_run[1] += __shfl_xor_sync(0xffffffffu, l_run[1], 1);
    l_run[1] += __shfl_xor_sync(0xffffffffu, l_run[1], 2);
    cp_async_wait<0>();                                  // a CTA without rows still has its Q copy in flight
    __syncthreads();
    float* loc = reinterpret_cast<float*>(kv_s);        // [kvg][Tpad][REC], aliases the KV buffers
    if (active) {
        float* wo = loc + ((size_t)g * Tpad) * REC;
#pragma unroll
        for (int j = 0; j < NT; ++j) {
            int col = j * 8 + (lane & 3) * 2;
            *reinterpret_cast<float2*>(wo + (size_t)row_a * REC + col) = make_float2(o[j][0], o[j][1]);
            *reinterpret_cast<float2*>(wo + (size_t)row_b * REC + col) = make_float2(o[j][2], o[j][3]);
        }
        if ((lane & 3) == 0) {
            *reinterpret_cast<float2*>(wo + (size_t)row_a * REC + HD) = make_float2(m_run[0], l_run[0]);
            *reinterpret_cast<float2*>(wo + (size_t)row_b * REC + HD) = make_float2(m_run[1], l_run[1]);
        }
    }
    const int csize = p.csize, rpr = p.rpr;
    const int rank = split % csize, outer = split / csize;
    const int n_parts = csize * p.kvg;                         // <= 32
    const float* src_parts = loc;                              // csize == 1: merge straight from the deposit
    int part_stride = Tpad * REC, row0 = 0, n_my = Tpad;
    if (csize > 1) {
        asm volatile("fence.proxy.async.shared::cta;" ::: "memory");   // the deposit is read by bulk copies
        __syncthreads();
        // one thread per (destination, g) sends slab g of the rows that destination owns; a bulk copy occupies its
        // issuing thread for about half a microsecond, so the senders are spread over the warps
        const int pi = lane * 8 + warp;
        if (lane < 4 && pi < n_parts) {
            const int dest = pi / p.kvg, gg = pi - dest * p.kvg;
            const int r0 = min(Tpad, dest * rpr), r1 = min(Tpad, r0 + rpr);
            if (r1 > r0) {
                const uint32_t bytes = (uint32_t)(r1 - r0) * REC * 4;
                const uint32_t src = smem_u32(loc + ((size_t)gg * Tpad + r0) * REC);
                const uint32_t dst_local = smem_u32(recv + ((size_t)(rank * p.kvg + gg) * rpr) * REC);
                const uint32_t dst = cluster_map(dst_local, dest), bar = cluster_map(smem_u32(rbar), dest);
                asm volatile("cp.async.bulk.shared::cluster.shared::cta.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];"
                             ::"r"(dst), "r"(src), "r"(bytes), "r"(bar) : "memory");
            }
        }
        row0 = min(Tpad, rank * rpr);
        n_my = min(Tpad, row0 + rpr) - row0;
        if (n_my > 0 && !mbar_wait(rbar, 0, wait_expired)) {
            if (threadIdx.x == 0) report(p.d_status, CATS_ERR_TIMEOUT);
        }
        asm volatile("barrier.cluster.arrive.release.aligned;" ::: "memory");   // this CTA holds everything it needs
        src_parts = recv;
        part_stride = rpr * REC;
    } else {
        __syncthreads();
    }
    for (int rl = warp; rl < n_my; rl += 8) {
        const int row = row_base + row0 + rl;      // global query row
        if (row >= p.T) break;
        float mp = -INFINITY, lp = 0.f;
        const float* my_rec = src_parts;
        if (lane < n_parts) {
            my_rec = src_parts + (size_t)lane * part_stride + (size_t)(csize > 1 ? rl : row0 + rl) * REC;
            const float2 ml = *reinterpret_cast<const float2*>(my_rec + HD);
            mp = ml.x; lp = ml.y;
        }
        float M = mp;
#pragma unroll
        for (int ofs = 16; ofs > 0; ofs >>= 1) M = fmaxf(M, __shfl_xor_sync(0xffffffffu, M, ofs));
        const float ref = (M == -INFINITY) ? 0.f : M;
        const float wp = exp2f(mp - ref);
        float L = lp * wp;
#pragma unroll
        for (int ofs = 16; ofs > 0; ofs >>= 1) L += __shfl_xor_sync(0xffffffffu, L, ofs);
        float4 acc = make_float4(0.f, 0.f, 0.f, 0.f);
        const bool col_ok = lane < HD / 4;
        const float* base = src_parts + (size_t)(csize > 1 ? rl : row0 + rl) * REC + lane * 4;
        for (int pp = 0; pp < n_parts; ++pp) {                 // partials in a fixed order
            const float w = __shfl_sync(0xffffffffu, wp, pp);
            if (col_ok && w != 0.f) {
                const float4 v = *reinterpret_cast<const float4*>(base + (size_t)pp * part_stride);
                acc.x += v.x * w; acc.y += v.y * w; acc.z += v.z * w; acc.w += v.w * w;
            }
        }
        if (p.n_outer == 1) {
            if (col_ok) {
                const float inv = 1.f / L;
                uint2 pk = make_uint2(pack_bf16x2(acc.x * inv, acc.y * inv), pack_bf16x2(acc.z * inv, acc.w * inv));
                uint8_t* ob = reinterpret_cast<uint8_t*>(p.out);
                const int col = lane * 4;
                size_t off = p.out_npad > 0 ? packed_act_offset(row, (h * HD + col) >> 3, p.out_npad) + (size_t)(col & 7) * 2
                                            : (((size_t)row * p.nh + h) * HD + col) * 2;
                *reinterpret_cast<uint2*>(ob + off) = pk;
            }
        } else {
            const size_t gbase = ((size_t)h * p.n_outer + outer) * Tpad + row;
            if (col_ok) *reinterpret_cast<float4*>(p.part_o + gbase * HD + lane * 4) = acc;
            if (lane == 0) { p.part_ml[gbase * 2] = M; p.part_ml[gbase * 2 + 1] = L; }
        }
    }
    // nobody leaves while a peer's copy may still be reading this CTA's deposit
    if (csize > 1) asm volatile("barrier.cluster.wait.acquire.aligned;" ::: "memory");
}

// ---------------------------------------------------------------------------------------------------
// The same attention on the 5th-generation tensor cores (head_dim 128).
//
// One CTA per (head, share of the cache rows), ten or eleven warps.  Q (128 rows, zero beyond T) and a ring of K/V
// blocks sit in shared memory in the layout tcgen05.mma reads: two halves of 64 head-dim elements, each a stack of
// 128-byte rows with the 128-byte swizzle, written by TMA (one thread of warp 9 issues every copy; a refill goes into
// the stage the last P V product released).  The SAME bytes serve as the K-major operand of S = Q K^T (row = cache
// row) and as the MN-major operand of O += P V (row = K index).  One thread of warp 8 issues S(b) = Q K(b)^T as soon
// as block b has landed (and the product that read the S / P buffer of block b - 2 has completed), one thread of
// warp 10 issues P(b) V(b) as soon as P(b) is written: the tensor core works on the next block during the softmax of
// this one, and neither kind of product waits for the ~100 cycles the other's issue costs per instruction.
// S has two buffers in tensor memory, one query row per lane; warps w and w+4 share the 32 rows of lane quadrant
// w and split the block's columns.  The reference of the exponentials moves only when a row's maximum outgrows it
// by 2^8, which the two warps find out by a vote inside the barrier that orders their loads of S before their stores
// of P; only then are maxima exchanged and O (in tensor memory) rescaled.  The probabilities go back to tensor
// memory over the columns S occupied, as two bf16 operands hi + lo (the upper and the next 16 bits of the fp32
// value), and enter P V as the A operand from tensor memory.  The CTA's partial (m, l, O) is then merged across the
// cluster: every softmax thread stores its half row straight into the shared memory of the CTA that merges that row
// (distributed shared memory; one phase of the cluster barrier makes sure every CTA has started, the next publishes the
// records), and the merge reads local memory only.  A share of at most 192 rows is one block: those instances are compiled without ring, vote, rescale
// and second issuing warp (warp 8 issues both products).
// ---------------------------------------------------------------------------------------------------
constexpr int kTcThreads = 352;       // warps 0-7: softmax; 8: issue of Q K^T, tensor-memory allocation; 9: TMA loads; 10: issue of P V
                                      // (streamed shares only: a one-block share is launched with 320 threads)
// Trees of at most 64 nodes fill only the tensor-memory lanes 0-63, which only warps with (warp index mod 4) in {0, 1} can
// reach: the WIDE instances run 14 warps so that eight of them (0, 1, 4, 5, 8, 9, 12, 13) are such warps and FOUR threads
// share every query row instead of two.  There warp 2 issues Q K^T and allocates, warp 3 loads, warp 6 issues P V.
// Larger trees get four threads per row too, with sixteen softmax warps (0-15; 16 issues Q K^T, 17 loads, 18 issues
// P V): 19 warps leave 104 registers per thread, enough for every instance (at most 48 columns of S per thread: 87).
constexpr int kTcThreadsWide = 448;
constexpr int kTcThreadsWide128 = 608;
constexpr int tc_threads(int wd) { return wd == 0 ? kTcThreads : (wd == 1 ? kTcThreadsWide : kTcThreadsWide128); }
constexpr int kTcBoxRows = 32;        // rows of one TMA box (64 head-dim elements wide)
constexpr int kTcCols = 512;          // tensor-memory columns: S0 / P [0,192), S1 / P [192,384), O [384,512)
constexpr int kTcSStride = 192;
constexpr int kTcStream = 64;         // cache rows per block when a share is streamed
constexpr int kTcOneShot = 192;       // a share of at most this many rows is one block
constexpr int kTcMaxStages = 7;

__device__ __forceinline__ void tmem_ld16_nowait(uint32_t taddr, float* v) {
    uint32_t r[16];
    asm volatile(
        "tcgen05.ld.sync.aligned.32x32b.x16.b32 {%0, %1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15}, [%16];"
        : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7]), "=r"(r[8]),
          "=r"(r[9]), "=r"(r[10]), "=r"(r[11]), "=r"(r[12]), "=r"(r[13]), "=r"(r[14]), "=r"(r[15])
        : "r"(taddr)
        : "memory");
#pragma unroll
    for (int i = 0; i < 16; ++i) v[i] = __uint_as_float(r[i]);
}
// Completes the loads above; the values may be used only after the empty statements that tie them to this point.
template <int N>
__device__ __forceinline__ void tmem_wait_ld(float* v) {
    asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory");
#pragma unroll
    for (int i = 0; i < N; ++i) asm volatile("" : "+f"(v[i]));
}
__device__ __forceinline__ float ex2_approx(float x) {
    float y;
    asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
    return y;
}
// Bit e set iff cache row g0 + e is visible to the query whose ancestor mask is (m0, m1): prefix rows always, tree
// rows by their mask bit, nothing from c_end on.
__device__ __forceinline__ uint32_t tc_visible16(int g0, int P, int c_end, uint64_t m0, uint64_t m1) {
    const int np = min(max(min(P, c_end) - g0, 0), 16);
    uint32_t bits = (1u << np) - 1u;
    const int e0 = max(P - g0, 0);
    if (e0 < 16) {
        const int j0 = g0 + e0 - P;                       // first tree row of the group, 0 <= j0
        uint64_t w = 0ull;
        if (j0 < 64) w = (m0 >> j0) | (j0 > 0 ? (m1 << (64 - j0)) : 0ull);
        else if (j0 < 128) w = m1 >> (j0 - 64);
        const int nv = min(max(c_end - (g0 + e0), 0), 16);
        bits |= (((uint32_t)w & ((1u << nv) - 1u)) << e0) & 0xffffu;
    }
    return bits;
}
template <int NT>
__device__ __forceinline__ void pair_barrier(int quadrant) {     // the NT threads (two or four warps) that share a lane quadrant
    asm volatile("bar.sync %0, %1;" ::"r"(quadrant + 1), "n"(NT) : "memory");
}
template <int NT>
__device__ __forceinline__ bool pair_barrier_or(int quadrant, bool pred) {     // the same barrier, returning the OR of pred
    uint32_t r;
    asm volatile(
        "{\n\t.reg .pred p, q;\n\t"
        "setp.ne.b32 q, %1, 0;\n\t"
        "bar.red.or.pred p, %2, %3, q;\n\t"
        "selp.u32 %0, 1, 0, p;\n\t}"
        : "=r"(r)
        : "r"((uint32_t)pred), "r"(quadrant + 1), "n"(NT)
        : "memory");
    return r != 0;
}

// CPT: the most columns of S one softmax thread holds (a block has at most 2 CPT rows); instances for the streamed
// 64-row blocks and for one-block shares of up to 128, 160 and 192 rows.
// STREAM: the share is streamed in blocks (otherwise it is one block, and everything that hands blocks on is compiled out).
template <int CPT, bool STREAM, int WIDE>      // WIDE: 0 two softmax threads per query row, 1 four (trees of <= 64 nodes), 2 four (any tree)
__global__ void __launch_bounds__(tc_threads(WIDE), 1) k_tree_attn_tc(const AttnDev p, const __grid_constant__ CUtensorMap tm_q,
                                                                const __grid_constant__ CUtensorMap tm_k,
                                                                const __grid_constant__ CUtensorMap tm_v) {
    extern __shared__ __align__(128) uint8_t sm_raw[];
    constexpr int HD = 128, REC = HD + 4;
    if (threadIdx.x == 0) ATTN_TL(0);
    uint8_t* sm = sm_raw + ((1024u - (smem_u32(sm_raw) & 1023u)) & 1023u);      // the operand tiles need 1024-byte alignment
    const int Tpad = p.n_mt * 16;
    // Q holds only the 32-row boxes that contain rows of the batch; the MMA reads 128 rows per head-dim half all the same
    // (the rows beyond are whatever follows in shared memory; nobody reads their results).
    const int q_rows = (Tpad + kTcBoxRows - 1) / kTcBoxRows * kTcBoxRows;
    uint8_t* q_s = sm;                                                           // [2][q_rows][128 B]
    uint8_t* kv_s = q_s + (size_t)q_rows * 256;                                  // ring of K and V blocks
    constexpr int NH = WIDE ? 4 : 2;                                             // softmax threads per query row
    constexpr int W_ISSUE = WIDE == 0 ? 8 : (WIDE == 1 ? 2 : 16), W_LOAD = W_ISSUE + 1, W_PV = WIDE == 1 ? 6 : W_ISSUE + 2;
    constexpr int N_SOFTMAX = WIDE == 2 ? 512 : 256;                             // softmax threads (arrivals per hand-off)
    float* xch = reinterpret_cast<float*>(kv_s + p.kv_area);                    // [2][NH][128] row maxima (by block parity), [NH][128] row sums
    // The records the cluster's CTAs deposit here, [csize][rpr][REC].  Either an area of their own: then nothing but
    // "that CTA has started" is required before a peer stores into it, and every thread arrives at the cluster barrier
    // right after the set-up.  Or (recv_over_ring: streamed shares of large trees, where the area would cost two of five
    // ring stages) they lie over the ring: then every thread arrives only when its part of the streaming is over, which
    // costs the barrier's latency in front of the deposit.
    const bool over_ring = p.recv_over_ring != 0;
    float* recv = over_ring ? reinterpret_cast<float*>(kv_s) : xch + 3 * NH * 128;
    uint64_t* rbar = reinterpret_cast<uint64_t*>(xch + 3 * NH * 128 + ((p.csize > 1 && !over_ring) ? (size_t)p.csize * p.rpr * REC : 0));   // base of the mbarriers; slot 0 unused
    // Every barrier that a thread may find more than one phase ahead of itself would give a wrong answer to a parity
    // wait, so each one is either indexed by block parity (its next completion needs the waiter's own progress) or by
    // ring stage (the classical full / empty pair).
    // Streamed shares keep FOUR score / probability buffers in tensor memory (one-block shares use one): the loop
    // S(b) -> softmax -> P(b) V(b) -> buffer free again is a chain of three hand-offs of several hundred nanoseconds each,
    // and with two buffers that chain, not any unit's throughput, set the pace (halving the MMAs, the TMA issues or the
    // softmax work per thread each changed next to nothing).
    constexpr int NSB = STREAM ? 4 : 2;
    uint64_t* bar_s = rbar + 1;           // [4]  S(b) complete, by buffer (b mod NSB)
    uint64_t* bar_o = rbar + 5;           // [4]  P(b) V(b) complete, by buffer
    uint64_t* bar_p = rbar + 9;           // [4]  P(b) written (256 arrivals), by buffer
    uint64_t* bar_kv = rbar + 13;         // [kTcMaxStages]  block landed in the stage (bytes counted)
    uint64_t* bar_free = bar_kv + kTcMaxStages;  // [kTcMaxStages]  the P V product that read the stage has completed
    uint64_t* bar_q = bar_free + kTcMaxStages;   //      Q landed
    uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(bar_q + 1);
    volatile int* wait_expired = reinterpret_cast<volatile int*>(tmem_slot + 1);

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const bool softmax_warp = WIDE == 0 ? warp < 8 : (WIDE == 1 ? (warp & 2) == 0 : warp < 16);
    const int split = (int)blockIdx.x, h = blockIdx.y;
    const int S = p.P + p.Tk;
    const int c_begin = min(S, split * p.rows_per_split);
    const int c_end = min(S, c_begin + p.rows_per_split);
    const int NB = p.blk;                                  // rows per block, a multiple of 32
    const int NST = p.stages;                              // stages of the ring
    const int nb = STREAM ? (c_end - c_begin + NB - 1) / NB : (c_end > c_begin ? 1 : 0);
    const uint32_t half = (uint32_t)NB * 128u;             // bytes between the two head-dim halves of a block
    const size_t stage_bytes = (size_t)NB * 512;           // K block, then V block

    // One thread (warp 9) moves everything with TMA: boxes of 32 rows x 64 head-dim elements land as 32 swizzled
    // 128-byte rows.  The tensor maps end at row P + T_tree (K, V) and T (Q): rows beyond read as zeros.  Rows between
    // the end of this CTA's share and the end of the cache are another CTA's (finite values, masked in the softmax).
    // part 0: boxes wholly below the prefix length (no dependence on the previous kernel); 1: the others; 2: all.
    auto load_kv = [&](int b, int stage, int part, uint64_t policy) {
        uint8_t* ks = kv_s + (size_t)stage * stage_bytes;
        uint8_t* vs = ks + (size_t)NB * 256;
        const int r0 = c_begin + b * NB;
        for (int rb = 0; rb < NB; rb += kTcBoxRows) {
            const bool below = r0 + rb + kTcBoxRows <= p.P;
            if ((part == 0 && !below) || (part == 1 && below)) continue;
#pragma unroll
            for (int hh = 0; hh < 2; ++hh) {
                tma_load_2d(ks + (size_t)hh * half + (size_t)rb * 128, &tm_k, h * HD + hh * 64, r0 + rb, bar_kv + stage, policy);
                tma_load_2d(vs + (size_t)hh * half + (size_t)rb * 128, &tm_v, h * HD + hh * 64, r0 + rb, bar_kv + stage, policy);
            }
        }
    };

    pdl_launch_dependents();
    if (warp == W_ISSUE) {
        tmem_alloc(tmem_slot, kTcCols);
        tmem_relinquish();
        if (lane == 0) {
            *wait_expired = 0;
            for (int i = 0; i < NSB; ++i) {
                mbar_init(bar_s + i, 1);
                mbar_init(bar_o + i, 1);
                mbar_init(bar_p + i, N_SOFTMAX);
            }
            mbar_fence_init();
        }
    }
    uint64_t ld_policy = 0;
    if (warp == W_LOAD && lane == 0) {
        // The loader sets up its own barriers and requests the prefix rows of every stage of the ring at once: they depend
        // neither on the previous kernel nor on the rest of the set-up.
        for (int i = 0; i < kTcMaxStages; ++i) { mbar_init(bar_kv + i, 1); mbar_init(bar_free + i, 1); }
        mbar_init(bar_q, 1);
        mbar_fence_init();
        ld_policy = l2_policy_evict_first();
        for (int b = 0; b < NST && b < nb; ++b) {
            mbar_expect_tx(bar_kv + b, (uint32_t)stage_bytes);
            load_kv(b, b, 0, ld_policy);
        }
    }
    tc_fence_before_sync();
    __syncthreads();
    tc_fence_after_sync();
    if (threadIdx.x == 0) ATTN_TL(1);
    if (p.csize > 1 && !over_ring) asm volatile("barrier.cluster.arrive.release.aligned;" ::: "memory");
    pdl_wait();
    if (threadIdx.x == 0) ATTN_TL(2);
    const uint32_t tbase = *tmem_slot;
    // tensor-memory columns.  One-block share: S / P [0,192), O [384,512).  Streamed: S / P buffers [64 k, 64 k + 64), k < 4.
    const uint32_t tO = tbase + 384;
    auto sbuf = [&](int b) { return STREAM ? (b & 3) : (b & 1); };              // buffer of block b
    auto sphase = [&](int b) { return (uint32_t)(STREAM ? (b >> 2) : (b >> 1)) & 1u; };   // and the phase of its barriers
    auto s_addr = [&](int b) { return tbase + (uint32_t)(STREAM ? (b & 3) * 64 : (b & 1) * kTcSStride); };
    const uint32_t q_u32 = smem_u32(q_s);

    // O += P(b) V(b), issued as soon as the softmax warps have written P(b)
    auto issue_pv = [&](int b) -> bool {
        const uint32_t idv = umma_idesc_bf16_m128_bmn(HD);
        if (!(mbar_wait(bar_kv + b % NST, (uint32_t)(b / NST) & 1u, wait_expired) &&      // V(b) (long since landed)
              mbar_wait(bar_p + sbuf(b), sphase(b), wait_expired)))
            return false;
        tc_fence_after_sync();
        const int r0 = c_begin + b * NB;
        const int n16 = min(NB, (c_end - r0 + 15) & ~15);
        const uint32_t vs_u32 = smem_u32(kv_s + (size_t)(b % NST) * stage_bytes) + (uint32_t)NB * 256u;
        const uint32_t tP = s_addr(b);
        const uint64_t dv0 = umma_desc_sw128_mn(vs_u32, half);
        const int nk = n16 / 16;
        for (int kk = 0; kk < nk; ++kk)
            umma_bf16_ts(tO, tP + (uint32_t)kk * 8u, dv0 + (uint64_t)(kk * (2048 >> 4)), idv, b > 0 || kk > 0);
        for (int kk = 0; kk < nk; ++kk)
            umma_bf16_ts(tO, tP + (uint32_t)(NB / 2) + (uint32_t)kk * 8u, dv0 + (uint64_t)(kk * (2048 >> 4)), idv, true);
        umma_commit(bar_o + sbuf(b));
        umma_commit(bar_free + b % NST);
        return true;
    };
    if (warp == W_ISSUE) {
        // ---- issue of S(b) = Q K(b)^T: as soon as block b has landed and the product that read the S / P buffer of
        //      block b - 2 has completed (issuing one tcgen05.mma costs its thread about a hundred cycles, so the two
        //      kinds of products are issued by two threads) ----
        if (lane == 0 && nb > 0) {
            bool ok = mbar_wait(bar_q, 0, wait_expired);
            for (int b = 0; b < nb && ok; ++b) {
                ok = mbar_wait(bar_kv + b % NST, (uint32_t)(b / NST) & 1u, wait_expired);
                if (ok && b >= NSB) ok = mbar_wait(bar_o + sbuf(b), sphase(b - NSB), wait_expired);
                if (!ok) break;
                if (b == 0) ATTN_TL(4);
                tc_fence_after_sync();
                const int r0 = c_begin + b * NB;
                const int n16 = min(NB, (c_end - r0 + 15) & ~15);
                const uint32_t ks_u32 = smem_u32(kv_s + (size_t)(b % NST) * stage_bytes);
                const uint32_t tS = s_addr(b);
                const uint32_t idesc = umma_idesc_bf16_m128(n16);
                const uint64_t da0 = umma_desc_sw128(q_u32), db0 = umma_desc_sw128(ks_u32);      // the address field takes plain additions
#pragma unroll
                for (int ks = 0; ks < HD / 16; ++ks) {
                    const uint64_t da = da0 + (uint64_t)(((ks >> 2) * (q_rows * 128) + (ks & 3) * 32) >> 4);
                    const uint64_t db = db0 + (uint64_t)(((uint32_t)(ks >> 2) * half + (uint32_t)(ks & 3) * 32u) >> 4);
                    umma_bf16(tS, da, db, idesc, ks > 0);
                }
                umma_commit(bar_s + sbuf(b));
                if (b == 0) ATTN_TL(5);
            }
            if (!STREAM) {
                // A one-block share moves little data: HBM is free to fetch the coming projections' weights meanwhile.
                // Requested only now, when this CTA's own rows have landed: requests issued earlier queue up in front of
                // the cache rows of the CTAs that start last (measured: the kernel 3.8 us longer).
                const unsigned n_cta = gridDim.x * gridDim.y, me = blockIdx.y * gridDim.x + blockIdx.x;
#pragma unroll
                for (int w = 0; w < 3; ++w) l2_warm(p.warm[w], me, n_cta, 24);
            }
            if (!STREAM && ok) issue_pv(0);      // one-block share: the same thread issues P V as well
        }
    } else if (STREAM && warp == W_PV) {
        // ---- issue of O += P(b) V(b) for streamed shares (a one-block share is launched without this warp) ----
        if (lane == 0)
            for (int b = 0; b < nb; ++b)
                if (!issue_pv(b)) break;
    } else if (warp == W_LOAD) {
        // ---- loader: Q and the boxes that depend on the previous kernel, then a refill whenever a P V product frees a stage ----
        if (lane == 0) {
            if (nb > 0) mbar_expect_tx(bar_q, (uint32_t)q_rows * 256u);
            for (int rb = 0; rb < q_rows && nb > 0 && !p.dbg_skip_q; rb += kTcBoxRows) {
                tma_load_2d(q_s + (size_t)rb * 128, &tm_q, h * HD, rb, bar_q, ld_policy);
                tma_load_2d(q_s + (size_t)q_rows * 128 + (size_t)rb * 128, &tm_q, h * HD + 64, rb, bar_q, ld_policy);
            }
            for (int b = 0; b < NST && b < nb; ++b) load_kv(b, b, 1, ld_policy);
            ATTN_TL(3);
            for (int j = NST; STREAM && j < nb; ++j) {
                if (!mbar_wait(bar_free + j % NST, (uint32_t)(j / NST - 1) & 1u, wait_expired)) break;
                mbar_expect_tx(bar_kv + j % NST, (uint32_t)stage_bytes);
                load_kv(j, j % NST, 2, ld_policy);
            }
        }
    } else if (softmax_warp) {
        // ---- the eight softmax warps: NH of them share a lane quadrant and split the block's columns ----
        const int quad = warp & 3, hf = warp >> 2;
        const int row = quad * 32 + lane;                       // the query row (= TMEM lane) of this thread
        const bool act = quad * 32 < Tpad;                      // the warp owns query rows
        const uint32_t lane_base = (uint32_t)(quad * 32) << 16;
        const int ncol = ((NB / 16 + NH - 1) / NH) * 16, c0 = hf * ncol;   // this thread's columns of a block (whole groups of 16)
        uint64_t mk0 = 0ull, mk1 = 0ull;
        if (row < p.T) {
            const size_t node = p.nodes != nullptr ? p.nodes[row] : row;
            mk0 = p.mask[node * 2];
            mk1 = p.mask[node * 2 + 1];
        }
        float m_run = -INFINITY, l_run = 0.f;
        bool ok = true;
        for (int b = 0; b < nb; ++b) {
            const int r0 = c_begin + b * NB;
            const uint32_t tS = s_addr(b);
            float v[CPT];
            float corr = 1.f, ref = 0.f;
            if (ok) ok = mbar_wait(bar_s + sbuf(b), sphase(b), wait_expired);
            if (threadIdx.x == 0 && b == 0) ATTN_TL(6);
            tc_fence_after_sync();
            if (act) {
#pragma unroll
                for (int c = 0; c < CPT; c += 16)
                    if (c < ncol && c0 + c < NB) tmem_ld16_nowait(tS + lane_base + (uint32_t)(c0 + c), v + c);
                tmem_wait_ld<CPT>(v);
                const int lim = min(p.P, c_end);
                float mx4[4] = {-INFINITY, -INFINITY, -INFINITY, -INFINITY};      // independent chains
#pragma unroll
                for (int c = 0; c < CPT; c += 16) {
                    if (c < ncol && c0 + c < NB) {
                        const int g0 = r0 + c0 + c;
                        if (g0 + 16 > lim) {
                            const uint32_t vis = tc_visible16(g0, p.P, c_end, mk0, mk1);
#pragma unroll
                            for (int e = 0; e < 16; ++e) v[c + e] = ((vis >> e) & 1u) ? v[c + e] : -INFINITY;
                        }
#pragma unroll
                        for (int e = 0; e < 16; ++e) mx4[e & 3] = fmaxf(mx4[e & 3], v[c + e]);
                    }
                }
                float mx = fmaxf(fmaxf(mx4[0], mx4[1]), fmaxf(mx4[2], mx4[3])) * p.scale_log2;     // the scale is positive
                // The old reference is kept while the maximum grows by less than 2^8 (probabilities then stay below 256 and
                // nothing is rescaled); any reference gives the same merged result.  The two warps of a quadrant vote in the
                // barrier that also orders their loads of S before their stores of P; only if some row of the 32 wants
                // a new reference are the maxima exchanged.
                if (!STREAM) {
                    // the only block: its maximum is the reference (one exchange, whose barrier orders the loads and stores)
                    xch[hf * 128 + row] = mx;
                    pair_barrier<32 * NH>(quad);
                    m_run = mx;
#pragma unroll
                    for (int k = 1; k < NH; ++k) m_run = fmaxf(m_run, xch[((hf + k) % NH) * 128 + row]);
                    ref = (m_run == -INFINITY) ? 0.f : m_run;
                } else {
                    const bool want = !(m_run != -INFINITY && mx <= m_run + 8.f);
                    if (pair_barrier_or<32 * NH>(quad, want)) {
                        xch[((b & 1) * NH + hf) * 128 + row] = mx;
                        pair_barrier<32 * NH>(quad);
#pragma unroll
                        for (int k = 1; k < NH; ++k) mx = fmaxf(mx, xch[((b & 1) * NH + (hf + k) % NH) * 128 + row]);
                        const float mn = (m_run != -INFINITY && mx <= m_run + 8.f) ? m_run : fmaxf(m_run, mx);
                        ref = (mn == -INFINITY) ? 0.f : mn;
                        corr = exp2f(m_run - ref);
                        m_run = mn;
                    } else {
                        ref = m_run;
                    }
                }
            }
            if (STREAM && b > 0 && act && __any_sync(0xffffffffu, corr != 1.f)) {
                // O follows the reference; P(b-1) V(b-1) must have completed first
                if (ok) ok = mbar_wait(bar_o + sbuf(b - 1), sphase(b - 1), wait_expired);
                tc_fence_after_sync();
                {
#pragma unroll
                    for (int c = 0; c < HD / NH; c += 16) {
                        float o[16];
                        tmem_ld16(tO + lane_base + (uint32_t)(hf * (HD / NH) + c), o);
#pragma unroll
                        for (int e = 0; e < 16; ++e) o[e] *= corr;
                        tmem_st16(tO + lane_base + (uint32_t)(hf * (HD / NH) + c), o);
                    }
                }
            }
            if (act) {
                float ls4[4] = {0.f, 0.f, 0.f, 0.f};                      // independent chains, summed in a fixed order
#pragma unroll
                for (int c = 0; c < CPT; c += 16) {
                    if (c < ncol && c0 + c < NB) {
                        uint32_t hi[8], lo[8];
#pragma unroll
                        for (int e = 0; e < 16; e += 2) {
                            const float x0 = ex2_approx(fmaf(v[c + e], p.scale_log2, -ref));
                            const float x1 = ex2_approx(fmaf(v[c + e + 1], p.scale_log2, -ref));
                            ls4[(e >> 1) & 3] += x0 + x1;
                            // hi = the upper 16 bits of x (exact in bf16), lo = the upper 16 bits of x - hi: integer and
                            // byte-permute operations only, the conversion unit is left to the exponentials
                            const uint32_t b0 = __float_as_uint(x0), b1 = __float_as_uint(x1);
                            hi[e >> 1] = __byte_perm(b0, b1, 0x7632);
                            const float l0 = x0 - __uint_as_float(b0 & 0xffff0000u), l1 = x1 - __uint_as_float(b1 & 0xffff0000u);
                            lo[e >> 1] = __byte_perm(__float_as_uint(l0), __float_as_uint(l1), 0x7632);
                        }
                        tmem_st8(tS + lane_base + (uint32_t)((c0 + c) >> 1), hi);
                        tmem_st8(tS + lane_base + (uint32_t)(NB / 2 + ((c0 + c) >> 1)), lo);
                    }
                }
                l_run = (STREAM ? l_run * corr : 0.f) + ((ls4[0] + ls4[1]) + (ls4[2] + ls4[3]));
                tmem_wait_st();
            }
            tc_fence_before_sync();
            // One hand-off barrier per buffer, counting one arrival per thread and block: no arrival for block b can come
            // before every thread has arrived for the buffer's previous block (S(b) is issued only after that block's
            // P V has completed, which needed all of its P).
            mbar_arrive(bar_p + sbuf(b));
            if (threadIdx.x == 0 && b == nb - 1) ATTN_TL(7);
        }
        // ---- this thread's half of the row's O, and the row's (m, l), go straight into the shared memory of the CTA
        //      that merges the row: stores through distributed shared memory, made visible by the cluster barrier ----
        if (nb > 0) {
            if (ok) ok = mbar_wait(bar_o + sbuf(nb - 1), sphase(nb - 1), wait_expired);
            tc_fence_after_sync();
        }
        if (threadIdx.x == 0) ATTN_TL(8);
        // Nobody stores into a peer's shared memory before that CTA has started, or, with the records over the ring, is done
        // with its ring: the first phase of the cluster barrier (over_ring: these warps arrive now that their last product
        // has completed, the others when they have issued their last copy or MMA).
        if (p.csize > 1 && over_ring) asm volatile("barrier.cluster.arrive.release.aligned;" ::: "memory");
        if (p.csize > 1) asm volatile("barrier.cluster.wait.acquire.aligned;" ::: "memory");
        if (act) {
            float* xl = xch + 2 * NH * 128;                     // [NH][128]
            xl[hf * 128 + row] = l_run;
            // the record of (part = this CTA, row): in the merging CTA's recv area, or, for a lone CTA, over the idle ring
            const int dest = p.csize > 1 ? min(row / p.rpr, p.csize - 1) : 0;
            const float* rec = p.csize > 1 ? recv + ((size_t)(split % p.csize) * p.rpr + (row - dest * p.rpr)) * REC
                                           : reinterpret_cast<const float*>(kv_s) + (size_t)row * REC;
            const uint32_t ra = cluster_map(smem_u32(rec), dest);
#pragma unroll
            for (int c = 0; c < HD / NH; c += 16) {
                float o[16];
                if (nb > 0) {
                    tmem_ld16(tO + lane_base + (uint32_t)(hf * (HD / NH) + c), o);
                } else {
#pragma unroll
                    for (int e = 0; e < 16; ++e) o[e] = 0.f;
                }
                if (row < Tpad) {
#pragma unroll
                    for (int e = 0; e < 16; e += 4)
                        asm volatile("st.shared::cluster.v4.f32 [%0], {%1, %2, %3, %4};"
                                     ::"r"(ra + (uint32_t)(hf * (HD / NH) + c + e) * 4u), "f"(o[e]), "f"(o[e + 1]), "f"(o[e + 2]), "f"(o[e + 3]) : "memory");
                }
            }
            pair_barrier<32 * NH>(quad);
            if (hf == 0 && row < Tpad) {
                float l_tot = l_run;
#pragma unroll
                for (int k = 1; k < NH; ++k) l_tot += xl[k * 128 + row];
                asm volatile("st.shared::cluster.v2.f32 [%0], {%1, %2};" ::"r"(ra + (uint32_t)HD * 4u), "f"(m_run), "f"(l_tot) : "memory");
            }
        }
    }
    if (threadIdx.x == 0) ATTN_TL(9);
    tc_fence_before_sync();
    const int csize = p.csize, rpr = p.rpr;
    const int rank = split % csize, outer = split / csize;
    const int n_parts = csize;
    const float* src_parts = reinterpret_cast<const float*>(kv_s);
    int part_stride = Tpad * REC, row0 = 0, n_my = Tpad;
    if (csize > 1) {
        // the softmax warps have passed the first phase of the cluster barrier above; the second one publishes the records
        if (!softmax_warp && over_ring) asm volatile("barrier.cluster.arrive.release.aligned;" ::: "memory");
        if (!softmax_warp) asm volatile("barrier.cluster.wait.acquire.aligned;" ::: "memory");
        asm volatile("barrier.cluster.arrive.release.aligned;" ::: "memory");
        asm volatile("barrier.cluster.wait.acquire.aligned;" ::: "memory");
        row0 = min(Tpad, rank * rpr);
        n_my = min(Tpad, row0 + rpr) - row0;
        src_parts = recv;
        part_stride = rpr * REC;
    } else {
        __syncthreads();
    }
    if (threadIdx.x == 0) ATTN_TL(10);
    if (warp == W_ISSUE) {
        tc_fence_after_sync();
        tmem_dealloc(tbase, kTcCols);
    }
    if (threadIdx.x == 0 && *wait_expired) report(p.d_status, CATS_ERR_TIMEOUT);
    // One thread per (query row, 8 output columns): all rows of the CTA are merged at once, every load of a thread is
    // independent of the others (the (m, l) pairs are broadcast reads), and the result leaves as one 16-byte store.
    for (int it = threadIdx.x; it < n_my * (HD / 8); it += (int)blockDim.x) {
        const int rl = it / (HD / 8), c8 = (it % (HD / 8)) * 8;
        const int grow = row0 + rl;                    // global query row
        if (grow >= p.T) continue;
        const float* rec0 = src_parts + (size_t)(csize > 1 ? rl : grow) * REC;
        float mpv[8], lpv[8], M = -INFINITY;
#pragma unroll
        for (int pp = 0; pp < 8; ++pp) {
            mpv[pp] = -INFINITY; lpv[pp] = 0.f;
            if (pp < n_parts) {
                const float2 ml = *reinterpret_cast<const float2*>(rec0 + (size_t)pp * part_stride + HD);
                mpv[pp] = ml.x; lpv[pp] = ml.y;
                M = fmaxf(M, ml.x);
            }
        }
        const float ref = (M == -INFINITY) ? 0.f : M;
        float L = 0.f;
        float acc[8] = {0.f, 0.f, 0.f, 0.f, 0.f, 0.f, 0.f, 0.f};
#pragma unroll
        for (int pp = 0; pp < 8; ++pp) {                       // partials in a fixed order
            if (pp < n_parts) {
                const float w = exp2f(mpv[pp] - ref);
                L += lpv[pp] * w;
                if (w != 0.f) {
                    const float4 v0 = *reinterpret_cast<const float4*>(rec0 + (size_t)pp * part_stride + c8);
                    const float4 v1 = *reinterpret_cast<const float4*>(rec0 + (size_t)pp * part_stride + c8 + 4);
                    acc[0] += v0.x * w; acc[1] += v0.y * w; acc[2] += v0.z * w; acc[3] += v0.w * w;
                    acc[4] += v1.x * w; acc[5] += v1.y * w; acc[6] += v1.z * w; acc[7] += v1.w * w;
                }
            }
        }
        if (p.n_outer == 1) {
            const float inv = 1.f / L;
            const uint4 pk = make_uint4(pack_bf16x2(acc[0] * inv, acc[1] * inv), pack_bf16x2(acc[2] * inv, acc[3] * inv),
                                        pack_bf16x2(acc[4] * inv, acc[5] * inv), pack_bf16x2(acc[6] * inv, acc[7] * inv));
            uint8_t* ob = reinterpret_cast<uint8_t*>(p.out);
            const size_t off = p.out_npad > 0 ? packed_act_offset(grow, (h * HD + c8) >> 3, p.out_npad)
                                              : (((size_t)grow * p.nh + h) * HD + c8) * 2;
            *reinterpret_cast<uint4*>(ob + off) = pk;
        } else {
            const size_t gbase = ((size_t)h * p.n_outer + outer) * Tpad + grow;
            *reinterpret_cast<float4*>(p.part_o + gbase * HD + c8) = make_float4(acc[0], acc[1], acc[2], acc[3]);
            *reinterpret_cast<float4*>(p.part_o + gbase * HD + c8 + 4) = make_float4(acc[4], acc[5], acc[6], acc[7]);
            if (c8 == 0) { p.part_ml[gbase * 2] = M; p.part_ml[gbase * 2 + 1] = L; }
        }
    }
    if (threadIdx.x == 0) ATTN_TL(11);
}

// out[t][h][:] = sum_s 2^(m_s - M) O_s / sum_s 2^(m_s - M) l_s over the clusters of a head.  One CTA per (node, head).
__global__ void __launch_bounds__(128) k_attn_combine(const float* __restrict__ part_o, const float* __restrict__ part_ml,
                                                      int n_splits, int Tpad, int nh, int hd, uint16_t* __restrict__ out,
                                                      int out_npad) {
    pdl_launch_dependents();
    pdl_wait();
    const int t = blockIdx.x, h = blockIdx.y, d = threadIdx.x;
    float M = -INFINITY;
    for (int s = 0; s < n_splits; ++s) M = fmaxf(M, part_ml[(((size_t)h * n_splits + s) * Tpad + t) * 2]);
    float L = 0.f, acc = 0.f;
    for (int s = 0; s < n_splits; ++s) {
        size_t base = ((size_t)h * n_splits + s) * Tpad + t;
        float w = exp2f(part_ml[base * 2] - M);
        L += part_ml[base * 2 + 1] * w;
        if (d < hd) acc += part_o[base * hd + d] * w;
    }
    if (d < hd) {
        uint16_t v = float_to_bf16_bits(acc / L);
        if (out_npad > 0)
            *reinterpret_cast<uint16_t*>(reinterpret_cast<uint8_t*>(out) + packed_act_offset(t, (h * hd + d) >> 3, out_npad) +
                                         (size_t)(d & 7) * 2) = v;
        else
            out[((size_t)t * nh + h) * hd + d] = v;
    }
}

// Chooses the cluster size (CTAs per head that share one merge through distributed shared memory) and, for long
// prefixes with few heads, the number of clusters per head.  Returns the bytes of workspace the outer merge needs.
// cats_debug_attention_kernel(0 / 1) forces the mma.sync / the tcgen05 kernel (for measurements and for testing the
// fallback); -1, the default: chosen by shape.
static int attn_tc_override() { return g_debug_attn_kernel; }
cudaError_t set_wait_limit_attn(unsigned long long ns) { return cudaMemcpyToSymbol(g_wait_limit_ns, &ns, sizeof(ns)); }

size_t attn_plan(AttnProblem& p) {
    const int S = p.prefix_len + (p.T_tree > 0 ? p.T_tree : p.T);
    const int units16 = (S + 15) / 16;
    const int tpad = ((p.T + 15) / 16) * 16;
    // as many CTAs per head as fit one wave of the 148 SMs (each CTA fills an SM), at most 8, at least 32 rows each
    int csize = 148 / p.nh;
    if (csize > 8) csize = 8;
    if (csize > units16 / 2) csize = units16 / 2;
    if (csize < 1) csize = 1;
    int n_outer = 1;
    int rows = (units16 + csize - 1) / csize * 16;
    if (p.nh * csize < 120 && rows > 128) {
        n_outer = (148 + p.nh * csize - 1) / (p.nh * csize);
        if (n_outer > rows / 128) n_outer = rows / 128;
        if (n_outer < 1) n_outer = 1;
    }
    // Trees of four or more query tiles over a short cache (<= 1024 rows): split the QUERY tiles over the CTAs of a head instead.
    // Every CTA then reads all cache rows of its head (the copies after the first come from L2), its eight warps
    // split each block of rows, and it finishes its own query rows alone: no exchange between CTAs at all.
    p.qsplit = 0;
    p.mt_per_cta = 0;
    // The tcgen05 kernel takes every head_dim-128 problem with a positive scale (measured in the 7B forward at prefix 512
    // against the mma.sync kernel: 3.07 vs 3.07 ms at T = 1, 3.09 vs 3.10 at 8, 3.11 vs 3.13 at 16, 3.15 vs 3.22 at 32,
    // 3.40 vs 3.48 at 64, 3.96 vs 4.14 at 128; alone over 16384 rows: 74 vs 81 us at T = 16, 85 vs 253 us at T = 128).
    p.use_tc = (p.hd == 128 && p.scale > 0.f) ? 1 : 0;
    if (attn_tc_override() >= 0) p.use_tc = (p.hd == 128 && p.scale > 0.f && attn_tc_override() >= 1) ? 1 : 0;
    const int n_mt = tpad / 16;
    if (!p.use_tc && n_mt >= 4 && S <= 1024) {     // measured at 32 heads: ahead up to about 1000 rows (15.8 vs 17.4 us at 576 rows), behind beyond
        int mpc = 1, groups = n_mt;
        if (p.nh * groups > 148) { mpc = 2; groups = (n_mt + 1) / 2; }
        if (p.nh * groups <= 148 && p.nh * groups >= 96) {
            p.qsplit = groups;
            p.mt_per_cta = mpc;
            p.n_splits = 1;
            p.cluster = 1;
            p.rows_per_split = units16 * 16;
            return 0;
        }
    }
    const int splits = csize * n_outer;
    p.n_splits = n_outer;
    p.cluster = csize;
    p.rows_per_split = (units16 + splits - 1) / splits * 16;
    return n_outer > 1 ? (size_t)p.nh * n_outer * tpad * (p.hd + 2) * sizeof(float) : 0;
}

template <typename Kern, typename... Extra>
static cudaError_t launch_cluster(Kern kernel, dim3 grid, dim3 block, size_t smem, int csize, cudaStream_t st, const AttnDev& d,
                                  const Extra&... extra) {
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = grid;
    cfg.blockDim = block;
    cfg.dynamicSmemBytes = smem;
    cfg.stream = st;
    cudaLaunchAttribute attr[2];
    int n = 0;
    attr[n].id = cudaLaunchAttributeClusterDimension;
    attr[n].val.clusterDim.x = (unsigned)csize;
    attr[n].val.clusterDim.y = 1;
    attr[n].val.clusterDim.z = 1;
    ++n;
    if (!g_call_boundary) {
        attr[n].id = cudaLaunchAttributeProgrammaticStreamSerialization;
        attr[n].val.programmaticStreamSerializationAllowed = 1;
        ++n;
    }
    g_call_boundary = false;
    cfg.attrs = attr;
    cfg.numAttrs = n;
    ++g_launch_count;
    return cudaLaunchKernelEx(&cfg, kernel, d, extra...);
}

// ---- tensor maps for the tcgen05 kernel ----------------------------------------------------------
// A [rows][cols] bf16 matrix with a row pitch, read in boxes of kTcBoxRows rows x 64 columns with the 128-byte swizzle;
// rows from `rows` on read as zeros.  The driver entry point is looked up once; the encoded maps are cached by
// (pointer, shape), since a decoding loop asks for the same few maps again and again.
typedef CUresult (*TensorMapEncodeFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*, const cuuint64_t*,
                                      const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave, CUtensorMapSwizzle,
                                      CUtensorMapL2promotion, CUtensorMapFloatOOBfill);
static TensorMapEncodeFn tensor_map_encoder() {
    static const TensorMapEncodeFn fn = [] {
        void* f = nullptr;
        cudaDriverEntryPointQueryResult q;
        if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &f, cudaEnableDefault, &q) != cudaSuccess || q != cudaDriverEntryPointSuccess)
            f = nullptr;
        return (TensorMapEncodeFn)f;
    }();
    return fn;
}
static bool attn_tensor_map(const void* ptr, long long cols, long long rows, long long pitch_elems, CUtensorMap* out) {
    struct Entry { const void* ptr; long long cols, rows, pitch; CUtensorMap map; bool used; };
    constexpr int kSlots = 256;
    static Entry cache[kSlots];
    static std::mutex mu;
    const size_t hsh = ((size_t)ptr >> 4) * 0x9E3779B97F4A7C15ull + (size_t)rows * 0xC2B2AE3D27D4EB4Full + (size_t)pitch_elems;
    Entry& e = cache[(hsh >> 20) % kSlots];
    std::lock_guard<std::mutex> lock(mu);
    if (e.used && e.ptr == ptr && e.cols == cols && e.rows == rows && e.pitch == pitch_elems) {
        *out = e.map;
        return true;
    }
    TensorMapEncodeFn enc = tensor_map_encoder();
    if (enc == nullptr) return false;
    const cuuint64_t dims[2] = {(cuuint64_t)cols, (cuuint64_t)rows};
    const cuuint64_t strides[1] = {(cuuint64_t)pitch_elems * 2};
    const cuuint32_t box[2] = {64, (cuuint32_t)kTcBoxRows};
    const cuuint32_t estr[2] = {1, 1};
    if (enc(&e.map, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, const_cast<void*>(ptr), dims, strides, box, estr, CU_TENSOR_MAP_INTERLEAVE_NONE,
            CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_128B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) != CUDA_SUCCESS) {
        e.used = false;
        return false;
    }
    e.ptr = ptr; e.cols = cols; e.rows = rows; e.pitch = pitch_elems; e.used = true;
    *out = e.map;
    return true;
}

// Returns cudaErrorNotSupported when the tensor maps cannot be made (the caller then uses the mma.sync kernel).
static cudaError_t launch_tree_attention_tc(const AttnProblem& p, cudaStream_t st) {
    static bool attr_set = false;
    if (!attr_set) {
        cudaError_t e = cudaFuncSetAttribute(k_tree_attn_tc<32, true, 0>, cudaFuncAttributeMaxDynamicSharedMemorySize, 227 * 1024);
        if (e == cudaSuccess) e = cudaFuncSetAttribute(k_tree_attn_tc<32, false, 0>, cudaFuncAttributeMaxDynamicSharedMemorySize, 227 * 1024);
        if (e == cudaSuccess) e = cudaFuncSetAttribute(k_tree_attn_tc<64, false, 0>, cudaFuncAttributeMaxDynamicSharedMemorySize, 227 * 1024);
        if (e == cudaSuccess) e = cudaFuncSetAttribute(k_tree_attn_tc<80, false, 0>, cudaFuncAttributeMaxDynamicSharedMemorySize, 227 * 1024);
        if (e == cudaSuccess) e = cudaFuncSetAttribute(k_tree_attn_tc<96, false, 0>, cudaFuncAttributeMaxDynamicSharedMemorySize, 227 * 1024);
        if (e == cudaSuccess) e = cudaFuncSetAttribute(k_tree_attn_tc<16, true, 1>, cudaFuncAttributeMaxDynamicSharedMemorySize, 227 * 1024);
        if (e == cudaSuccess) e = cudaFuncSetAttribute(k_tree_attn_tc<16, false, 1>, cudaFuncAttributeMaxDynamicSharedMemorySize, 227 * 1024);
        if (e == cudaSuccess) e = cudaFuncSetAttribute(k_tree_attn_tc<32, false, 1>, cudaFuncAttributeMaxDynamicSharedMemorySize, 227 * 1024);
        if (e == cudaSuccess) e = cudaFuncSetAttribute(k_tree_attn_tc<48, false, 1>, cudaFuncAttributeMaxDynamicSharedMemorySize, 227 * 1024);
        if (e == cudaSuccess) e = cudaFuncSetAttribute(k_tree_attn_tc<16, true, 2>, cudaFuncAttributeMaxDynamicSharedMemorySize, 227 * 1024);
        if (e == cudaSuccess) e = cudaFuncSetAttribute(k_tree_attn_tc<16, false, 2>, cudaFuncAttributeMaxDynamicSharedMemorySize, 227 * 1024);
        if (e == cudaSuccess) e = cudaFuncSetAttribute(k_tree_attn_tc<32, false, 2>, cudaFuncAttributeMaxDynamicSharedMemorySize, 227 * 1024);
        if (e == cudaSuccess) e = cudaFuncSetAttribute(k_tree_attn_tc<48, false, 2>, cudaFuncAttributeMaxDynamicSharedMemorySize, 227 * 1024);
        if (e != cudaSuccess) return e;
        attr_set = true;
    }
    AttnDev d;
    d.q = (const uint16_t*)p.q; d.k = (const uint16_t*)p.k; d.v = (const uint16_t*)p.v;
    d.mask = p.mask;
    d.nodes = p.nodes;
    d.Tk = p.T_tree > 0 ? p.T_tree : p.T;
    d.T = p.T; d.P = p.prefix_len; d.nh = p.nh;
    d.n_mt = (p.T + 15) / 16;
    d.kvg = 1;
    d.qsplit = 0;
    d.csize = p.cluster; d.n_outer = p.n_splits; d.rows_per_split = p.rows_per_split;
    d.kv_stride = p.kv_stride;
    d.scale_log2 = p.scale * 1.4426950408889634f;
    d.out = (uint16_t*)p.out;
    d.out_npad = p.out_packed_npad;
    d.part_o = p.part_o; d.part_ml = p.part_ml;
    d.d_status = p.d_status;
    d.dbg_skip_q = g_debug_fault == 2 ? 1 : 0;
#ifdef CATS_TIMELINE
    {
        unsigned long long* base = nullptr;
        cudaGetSymbolAddress((void**)&base, g_tl_attn);
        d.tl = base + (size_t)(g_tl_attn_next++ % 128) * kTlCtas * kTlStamps;
    }
#endif
    for (int w = 0; w < 3; ++w) d.warm[w] = warm_req(p.warm[w].ptr, p.warm[w].bytes, p.warm[w].period, p.warm[w].phase);
    const int tpad = d.n_mt * 16, rec = p.hd + 4;
    d.rpr = (((tpad + p.cluster - 1) / p.cluster) + 1) / 2 * 2;
    const size_t recv = p.cluster > 1 ? (size_t)p.cluster * d.rpr * rec * 4 : 0;
    // four softmax threads per query row (see kTcThreadsWide), on 8 softmax warps for trees of <= 64 nodes, else on 16
    const int wide = g_debug_attn_kernel == 2 ? 0 : (tpad <= 64 ? 1 : 2);
    const size_t q_bytes = (size_t)((tpad + kTcBoxRows - 1) / kTcBoxRows * kTcBoxRows) * 256;
    d.recv_over_ring = (p.cluster > 1 && wide == 2 && p.rows_per_split > kTcOneShot) ? 1 : 0;
    const size_t fixed = 1024 + q_bytes + (wide ? 6144 : 3072) + (d.recv_over_ring ? 0 : recv) + 320;     // alignment slack, Q, exchange among a row's threads, received records, barriers
    // the ring: stages of 64 rows of K and V (32 KB each), as many as fit, at least three (which also hold a one-block share)
    int stages = (int)((227 * 1024 - fixed) / (kTcStream * 512));
    if (stages > kTcMaxStages) stages = kTcMaxStages;
    if (stages < 3) return cudaErrorInvalidConfiguration;
    d.kv_area = stages * kTcStream * 512;
    if ((size_t)d.kv_area < (size_t)tpad * rec * 4 || (size_t)d.kv_area < recv) return cudaErrorInvalidConfiguration;   // the deposit lies over the ring
    if (p.rows_per_split <= kTcOneShot) {
        d.blk = (p.rows_per_split + 31) / 32 * 32;
        d.stages = 1;
    } else {
        d.blk = kTcStream;
        d.stages = stages;
    }
    const size_t smem = fixed + (size_t)d.kv_area;
    dim3 grid(p.cluster * p.n_splits, p.nh);
    CUtensorMap tm_q, tm_k, tm_v;
    const long long width = (long long)p.nh * p.hd;
    if (!attn_tensor_map(p.q, width, p.T, width, &tm_q) || !attn_tensor_map(p.k, width, p.prefix_len + d.Tk, p.kv_stride, &tm_k) ||
        !attn_tensor_map(p.v, width, p.prefix_len + d.Tk, p.kv_stride, &tm_v))
        return cudaErrorNotSupported;
    cudaError_t e;
    const dim3 one(kTcThreads - 32);      // the warp that issues P V on its own exists for streamed shares only
    const dim3 wd(kTcThreadsWide), wd2(kTcThreadsWide128);
    if (wide == 2) {
        if (d.stages > 1) e = launch_cluster(k_tree_attn_tc<16, true, 2>, grid, wd2, smem, p.cluster, st, d, tm_q, tm_k, tm_v);
        else if (d.blk <= 64) e = launch_cluster(k_tree_attn_tc<16, false, 2>, grid, wd2, smem, p.cluster, st, d, tm_q, tm_k, tm_v);
        else if (d.blk <= 128) e = launch_cluster(k_tree_attn_tc<32, false, 2>, grid, wd2, smem, p.cluster, st, d, tm_q, tm_k, tm_v);
        else e = launch_cluster(k_tree_attn_tc<48, false, 2>, grid, wd2, smem, p.cluster, st, d, tm_q, tm_k, tm_v);
    } else if (wide == 1) {
        if (d.stages > 1) e = launch_cluster(k_tree_attn_tc<16, true, 1>, grid, wd, smem, p.cluster, st, d, tm_q, tm_k, tm_v);
        else if (d.blk <= 64) e = launch_cluster(k_tree_attn_tc<16, false, 1>, grid, wd, smem, p.cluster, st, d, tm_q, tm_k, tm_v);
        else if (d.blk <= 128) e = launch_cluster(k_tree_attn_tc<32, false, 1>, grid, wd, smem, p.cluster, st, d, tm_q, tm_k, tm_v);
        else e = launch_cluster(k_tree_attn_tc<48, false, 1>, grid, wd, smem, p.cluster, st, d, tm_q, tm_k, tm_v);
    } else if (d.stages > 1) e = launch_cluster(k_tree_attn_tc<32, true, 0>, grid, dim3(kTcThreads), smem, p.cluster, st, d, tm_q, tm_k, tm_v);
    else if (d.blk <= 64) e = launch_cluster(k_tree_attn_tc<32, false, 0>, grid, one, smem, p.cluster, st, d, tm_q, tm_k, tm_v);
    else if (d.blk <= 128) e = launch_cluster(k_tree_attn_tc<64, false, 0>, grid, one, smem, p.cluster, st, d, tm_q, tm_k, tm_v);
    else if (d.blk <= 160) e = launch_cluster(k_tree_attn_tc<80, false, 0>, grid, one, smem, p.cluster, st, d, tm_q, tm_k, tm_v);
    else e = launch_cluster(k_tree_attn_tc<96, false, 0>, grid, one, smem, p.cluster, st, d, tm_q, tm_k, tm_v);
    if (e != cudaSuccess || p.n_splits == 1) return e;
    return launch_pdl(k_attn_combine, dim3(p.T, p.nh), dim3(128), 0, st, (const float*)p.part_o, (const float*)p.part_ml,
                      p.n_splits, tpad, p.nh, p.hd, (uint16_t*)p.out, p.out_packed_npad);
}

// Time line of the tcgen05 attention launches (measurement builds): copies the stamps to the host, or clears them.
cudaError_t timeline_attn(void* host, size_t bytes, bool clear) {
#ifdef CATS_TIMELINE
    if (clear) {
        void* b = nullptr;
        cudaError_t e = cudaGetSymbolAddress(&b, g_tl_attn);
        g_tl_attn_next = 0;
        return e != cudaSuccess ? e : cudaMemset(b, 0, sizeof(g_tl_attn));
    }
    return cudaMemcpyFromSymbol(host, g_tl_attn, bytes < sizeof(g_tl_attn) ? bytes : sizeof(g_tl_attn));
#else
    (void)host; (void)bytes; (void)clear;
    return cudaErrorNotSupported;
#endif
}

cudaError_t launch_tree_attention(const AttnProblem& p, cudaStream_t st) {
    static bool attr_set = false;
    if (!attr_set) {
        cudaError_t e = cudaFuncSetAttribute(k_tree_attn<128, false>, cudaFuncAttributeMaxDynamicSharedMemorySize, 227 * 1024);
        if (e == cudaSuccess) e = cudaFuncSetAttribute(k_tree_attn<128, true>, cudaFuncAttributeMaxDynamicSharedMemorySize, 227 * 1024);
        if (e == cudaSuccess) e = cudaFuncSetAttribute(k_tree_attn<64, false>, cudaFuncAttributeMaxDynamicSharedMemorySize, 227 * 1024);
        if (e == cudaSuccess) e = cudaFuncSetAttribute(k_tree_attn<64, true>, cudaFuncAttributeMaxDynamicSharedMemorySize, 227 * 1024);
        if (e != cudaSuccess) return e;
        attr_set = true;
    }
    if (p.use_tc) {
        const cudaError_t e = launch_tree_attention_tc(p, st);
        if (e != cudaErrorNotSupported) return e;     // no tensor maps on this driver: the kernel below takes any split
    }
    AttnDev d;
    d.q = (const uint16_t*)p.q; d.k = (const uint16_t*)p.k; d.v = (const uint16_t*)p.v;
    d.mask = p.mask;
    d.nodes = p.nodes;
    d.Tk = p.T_tree > 0 ? p.T_tree : p.T;
    d.T = p.T; d.P = p.prefix_len; d.nh = p.nh;
    d.n_mt = (p.T + 15) / 16;
    d.kvg = 8 / d.n_mt;
    if (d.kvg > 4) d.kvg = 4;
    if (d.kvg == 3) d.kvg = 2;
    d.qsplit = p.qsplit;
    if (p.qsplit > 0) {
        d.n_mt = p.mt_per_cta;       // query tiles per CTA
        d.kvg = 8 / d.n_mt;          // all eight warps split every block of cache rows
    }
    d.csize = p.cluster; d.n_outer = p.n_splits; d.rows_per_split = p.rows_per_split;
    d.kv_stride = p.kv_stride;
    d.scale_log2 = p.scale * 1.4426950408889634f;
    d.out = (uint16_t*)p.out;
    d.out_npad = p.out_packed_npad;
    d.part_o = p.part_o; d.part_ml = p.part_ml;
    int tpad = d.n_mt * 16;
    const int rec = p.hd + 4;
    size_t merge = (size_t)d.kvg * tpad * rec * 4;                  // the deposit aliases the KV buffers
    d.rpr = (((tpad + p.cluster - 1) / p.cluster) + 1) / 2 * 2;     // rows per CTA of the cluster, even
    d.d_status = p.d_status;
    const size_t recv = p.cluster > 1 ? (size_t)p.cluster * d.kvg * d.rpr * rec * 4 + 16 : 16;
    // Block size of the KV pipeline: a CTA whose whole share fits two or three 64-row blocks takes it in one block
    // instead (one wait and one barrier round instead of three); long shares stream 64-row blocks.
    int blk = kKvBlock;
    {
        const int gran = 16 * d.kvg;
        const int whole = (p.rows_per_split + gran - 1) / gran * gran;
        if (whole <= 192) blk = whole;
        if (p.qsplit > 0) blk = 128;   // one 16-row step per warp and block, double-buffered
    }
    d.blk = blk;
    const int n_buf = (p.rows_per_split <= blk) ? 1 : 2;            // a single block needs no second buffer
    size_t kv = (size_t)n_buf * 2 * blk * p.hd * 2;
    size_t qbytes = (size_t)tpad * p.hd * 2;                        // the (m, l) deposit area aliases Q
    if (qbytes < (size_t)d.kvg * tpad * 8) qbytes = (size_t)d.kvg * tpad * 8;
    if (kv < merge) kv = merge;
    d.kv_area = (int)kv;
    size_t smem = qbytes + kv + (size_t)tpad * 16 + recv;
    cudaError_t e;
    dim3 grid(p.qsplit > 0 ? p.qsplit : p.cluster * p.n_splits, p.nh);
    // a warp whose slice of a block has 32 rows or more takes prefix rows 32 at a time; the variant is compiled apart so
    // that the 16-row kernel keeps its register allocation
    const bool k32 = d.blk / d.kvg >= 32 && d.P >= 32;
    if (p.hd == 128) e = k32 ? launch_cluster(k_tree_attn<128, true>, grid, dim3(kAttnThreads), smem, p.cluster, st, d)
                             : launch_cluster(k_tree_attn<128, false>, grid, dim3(kAttnThreads), smem, p.cluster, st, d);
    else e = k32 ? launch_cluster(k_tree_attn<64, true>, grid, dim3(kAttnThreads), smem, p.cluster, st, d)
                 : launch_cluster(k_tree_attn<64, false>, grid, dim3(kAttnThreads), smem, p.cluster, st, d);
    if (e != cudaSuccess || p.n_splits == 1) return e;
    return launch_pdl(k_attn_combine, dim3(p.T, p.nh), dim3(128), 0, st, (const float*)p.part_o, (const float*)p.part_ml,
                      p.n_splits, tpad, p.nh, p.hd, (uint16_t*)p.out, p.out_packed_npad);
}

}  // namespace cats

// ---------------------------------------------------------------------------------------------------
// Allocation-free variant of cats_tree_attention.
//
// Some callers cannot hand the library a workspace because they cannot obtain device memory at the
// point of the call: code running between cudaStreamBeginCapture and EndCapture of someone else's
// graph, plugins that are given tensors but no allocator, latency-critical loops that must not touch
// the driver's allocator.  For them the split-KV partial results (running max, sum and unnormalised
// output per split) live in a fixed array inside the library image.  Every GPU that loads the library
// carries these CATS_STATIC_SCRATCH_BYTES until the process exits.
//
// g_attn_scratch is a device symbol: in host code its name is only a stand-in, not a device address.
// The address is looked up once per device with cudaGetSymbolAddress, with that device current, and
// that pointer is what the kernels receive.
// ---------------------------------------------------------------------------------------------------
namespace cats {
namespace {
constexpr size_t kStaticScratchBytes = CATS_STATIC_SCRATCH_BYTES;
static __device__ __align__(256) unsigned char g_attn_scratch[kStaticScratchBytes];
constexpr int kMaxDevices = 64;
void* g_attn_scratch_addr[kMaxDevices] = {};
std::mutex g_attn_scratch_mutex;

// Device address of the scratch array on the current device; looked up on the first call per device.
cudaError_t static_scratch_address(void** out) {
    int dev = -1;
    cudaError_t e = cudaGetDevice(&dev);
    if (e != cudaSuccess) return e;
    if (dev < 0 || dev >= kMaxDevices) return cudaErrorInvalidDevice;
    std::lock_guard<std::mutex> lock(g_attn_scratch_mutex);
    if (g_attn_scratch_addr[dev] == nullptr) {
        void* p = nullptr;
        e = cudaGetSymbolAddress(&p, g_attn_scratch);
        if (e != cudaSuccess) return e;
        if (p == nullptr) return cudaErrorInvalidSymbol;
        g_attn_scratch_addr[dev] = p;
    }
    *out = g_attn_scratch_addr[dev];
    return cudaSuccess;
}
}  // namespace
}  // namespace cats

extern "C" int cats_tree_attention_static(const void* d_q, const void* d_k, const void* d_v, const uint64_t* d_mask, int32_t T,
                                          int32_t prefix_len, int32_t n_heads, int32_t head_dim, int64_t kv_row_stride_elems,
                                          float scale, void* d_out, int32_t* d_status, void* stream) {
    using namespace cats;
    g_launch_count = 0;
    g_call_boundary = true;
    if (!d_q || !d_k || !d_v || !d_mask || !d_out || !d_status) return CATS_ERR_INVALID_ARG;
    if (T < 1 || T > CATS_MAX_TREE || prefix_len < 0 || n_heads < 1) return CATS_ERR_INVALID_ARG;
    if (head_dim != 64 && head_dim != 128) return CATS_ERR_UNSUPPORTED;
    if (kv_row_stride_elems < (int64_t)n_heads * head_dim || kv_row_stride_elems % 8) return CATS_ERR_INVALID_ARG;
    auto misaligned = [](const void* p, size_t a) { return (reinterpret_cast<uintptr_t>(p) % a) != 0; };
    if (misaligned(d_q, 16) || misaligned(d_k, 16) || misaligned(d_v, 16) || misaligned(d_out, 4)) return CATS_ERR_INVALID_ARG;
    AttnProblem a = {};
    a.q = d_q; a.k = d_k; a.v = d_v; a.mask = d_mask; a.T = T; a.prefix_len = prefix_len; a.nh = n_heads; a.hd = head_dim;
    a.kv_stride = kv_row_stride_elems; a.scale = scale; a.out = d_out; a.d_status = d_status;
    const size_t need = attn_plan(a);
    if (need > kStaticScratchBytes) return CATS_ERR_WORKSPACE;   // the problem needs more scratch than the library carries
    // Looked up on every call that passes the checks, whether or not this problem needs scratch, so that the FIRST
    // accepted call on a device always does the per-device set-up (a small warm-up call is enough).
    void* base = nullptr;
    if (static_scratch_address(&base) != cudaSuccess) return CATS_ERR_CUDA;
    if (need > 0) {
        const int tpad = (T + 15) / 16 * 16;
        a.part_o = static_cast<float*>(base);
        a.part_ml = a.part_o + (size_t)n_heads * a.n_splits * tpad * head_dim;
    }
    if (launch_tree_attention(a, (cudaStream_t)stream) != cudaSuccess) return CATS_ERR_CUDA;
    return CATS_OK;
}

