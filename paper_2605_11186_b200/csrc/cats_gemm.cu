// Skinny weight-streaming GEMM for the projections of the tree-verification forward.
//
//   Y^T[n_out, T] = W[n_out, K] * X^T[K, T]        (bf16 operands, fp32 accumulation, T <= 128)
//
// The problem is bound by reading W once from HBM, so everything is arranged around one contiguous
// read stream per SM:
//   * W is pre-packed (cats_pack_weights) into 16 KB chunks, one per (128-row tile, 64-column K block),
//     each chunk already in the shared-memory layout tcgen05.mma consumes (K-major rows of 128 bytes,
//     128-byte swizzle).  Chunks of a tile are consecutive, tiles are consecutive.
//   * X (the T tree nodes, padded to a multiple of 16) is kept by its producers in the same layout, one
//     chunk of n_pad x 128 bytes per K block.
//   * One persistent CTA per SM copies its share of the packed matrix with plain contiguous bulk copies, a
//     pattern that reaches the HBM copy rate.  How the (tile, K unit) pairs are shared out depends on the
//     projection (gemm_plan): aligned K pieces of every tile for the partial-sum projections, even contiguous
//     shares ("stream-K") when there are more tiles than SMs, one owner CTA per tile plus helper CTAs when
//     there are fewer.
// Warp 0 (one thread) copies W, warp 6 (one thread) copies X, both into a ring of shared-memory stages with
// mbarrier completion; warp 1 issues tcgen05.mma into one of two TMEM accumulators; warps 2-5 drain the other
// accumulator and run the epilogue.  A tile whose K range is shared by several CTAs is finished by the CTA
// that owns its first K units: the others publish fp32 partial tiles and a flag; the owner adds them in a fixed
// order (deterministic) and runs the epilogue.  Split-K partial sums of the O and down projections are
// not reduced here at all: the following RMSNorm kernel folds them into the residual stream.
//   EPI_PARTIAL  fp32 partial sums, one slot per piece of a tile
//   EPI_QKV      rotary embedding, bf16 q, k/v appended to the KV cache
//   EPI_SWIGLU   silu(gate) * up from a tile holding 64 gate rows and the matching 64 up rows
//   EPI_LMHEAD   fp32 logits, per-tile argmax candidates and (optionally) per-tile softmax statistics
// All epilogues go through a 32-node staging tile in shared memory so that every thread stores 16 bytes.
// Weight chunks of the first stages are requested before griddepcontrol.wait (weights never depend on
// an earlier kernel).  Every wait (mbarrier or flag) is bounded; on expiry the CTA reports
// CATS_ERR_TIMEOUT, lets its copies land, frees its TMEM and returns.
#include "cats_kernels.cuh"

namespace cats {

#ifndef CATS_GEMM_DUAL
#define CATS_GEMM_DUAL 1
#endif
constexpr int kGemmDualIssue = CATS_GEMM_DUAL;       // 1: two threads issue the MMAs (see mma_units)
constexpr int kGemmThreads = 384;      // warps: 0 W producer, 1 and 7 MMA issuers, 6 X producer, 2-5 and 8-11 epilogue groups
constexpr int kCtrlBytes = 512;
constexpr int kMaxStages = 14;
constexpr int kWChunk = 16384;        // 128 rows x 64 bf16
#ifndef CATS_UNIT_KB
#define CATS_UNIT_KB 2
#endif
constexpr int kUnitKb = CATS_UNIT_KB;   // K blocks per pipeline stage (one bulk copy of W, one of X)
constexpr int kStagingCols = 32;      // epilogue staging tile: 32 nodes x 128 features fp32

struct GemmDev {
    int epi, T, n_pad, n_out, n_kb, n_ku, n_tiles, tiles_per_mat, units_per_cta, n_stages, max_pieces, split_s;
    long long total_units;
    int head_units;       // > 0: "owners + helpers" split (see gemm_plan): CTA t < n_tiles runs units [0, head_units) of tile t
    int help_upc;         //   units per helper CTA in the space of the tiles' remaining units
    int total_rem;        //   n_tiles * (n_ku - head_units)
    uint32_t x_chunk_bytes, stage_bytes, tmem_cols;
    const uint8_t* Wp;
    const uint8_t* Xp;
    float* fix_part;      // [slots][n_pad][128] fp32 partial tiles of split tiles (slot = CTA, or 2 * tile + i with helpers)
    int* fix_flags;       // [slots]
    float* part;
    size_t part_stride;
    uint16_t *q_out, *kcache, *vcache;
    const float2* rope;
    int head_dim, prefix_len;
    const int32_t* kv_rows;
    uint8_t* act_out;     // packed activation layout
    float* logits;
    float* pmax;
    int32_t* pidx;
    float *psum, *ps1;            // EPI_LMHEAD, optional: per-tile softmax statistics [n_tiles][128]
    float inv_temp_log2e;         //   log2(e) / temperature
    const int32_t *tree_parent, *tree_tokens;   //   [T]
    float* cand;                  //   [T]: logit of every node's own token at its parent
    int32_t* d_status;
#ifdef CATS_TIMELINE
    unsigned long long* tl;      // this launch's time-line slot
#endif
    int dbg_skip_publish;        // fault injection: contributors of shared tiles keep their flags to themselves
};

#ifdef CATS_TIMELINE
#define GEMM_TL(slot) CATS_TL(p.tl, slot)
static __device__ unsigned long long g_tl_gemm[512 * kTlCtas * kTlStamps];
static int g_tl_gemm_next = 0;
#else
#define GEMM_TL(slot) do { } while (0)
#endif
// time-line stamps of this kernel: 0 CTA entered, 1 set-up done, 2 first weight copy issued, 3 first stage landed,
// 4 dependency resolved, 5 last weight copy issued, 6 last stage landed, 7 last accumulator complete, 8 epilogue done
// (group 0; 12: group 1), 9 CTA leaves, 10 the SM's id, 11 first activation copy issued

struct GemmCtrl {
    uint64_t full[kMaxStages];
    uint64_t empty[kMaxStages];
    uint64_t acc_full[2];
    uint64_t acc_empty[2];
    uint32_t tmem_base;
    int abort_flag;
};
static_assert(sizeof(GemmCtrl) <= kCtrlBytes, "control block too large");

constexpr int kEpiGroups = 2;         // groups of four epilogue warps (warps 2-5 and 8-11)
constexpr size_t kStagingBytes = (size_t)kEpiGroups * kStagingCols * 128 * 4;   // one staging tile per group
__device__ __forceinline__ void epi_barrier(int group) { asm volatile("bar.sync %0, 128;" ::"r"(group + 1) : "memory"); }
__device__ __forceinline__ void epi_barrier_all() { asm volatile("bar.sync 3, %0;" ::"n"(128 * kEpiGroups) : "memory"); }

__device__ __forceinline__ void bulk_load(void* smem_dst, const void* gsrc, uint32_t bytes, uint64_t* bar, uint64_t policy) {
    asm volatile(
        "cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes.L2::cache_hint [%0], [%1], %2, [%3], %4;"
        ::"r"(smem_u32(smem_dst)), "l"(gsrc), "r"(bytes), "r"(smem_u32(bar)), "l"(policy)
        : "memory");
}

// The accumulator tile of this CTA (thread = feature row f, columns = nodes) to global rows of 128 consecutive features
// per node: dst + node * row_stride + [0, 128).  Transposed through the staging tile, 32 nodes at a time, so that every
// store instruction of a warp writes 512 contiguous bytes (a quarter of the store instructions of the direct way, which
// was measured to be what the partial-sum epilogues were waiting for).  n_valid nodes, feat_limit: features that exist.
// 16 accumulator columns of this thread's row.  dual > 0: the sum was accumulated in two halves by two issuing threads
// (columns taddr and taddr + dual); they are added here, first half + second half.
__device__ __forceinline__ void acc_ld16(uint32_t taddr, uint32_t dual, float* v) {
    tmem_ld16(taddr, v);
    if (dual != 0) {
        float w[16];
        tmem_ld16(taddr + dual, w);
#pragma unroll
        for (int i = 0; i < 16; ++i) v[i] += w[i];
    }
}

__device__ __forceinline__ void store_tile_transposed(uint32_t taddr, uint32_t dual, int n_pad, int n_valid, float* acc_s, int f, int et,
                                                      int group, float* dst, size_t row_stride, int feat_limit) {
    for (int c0 = group * kStagingCols; c0 < n_valid; c0 += kEpiGroups * kStagingCols) {
#pragma unroll
        for (int hc = 0; hc < kStagingCols / 16; ++hc) {
            if (c0 + hc * 16 >= n_pad) break;
            float v[16];
            acc_ld16(taddr + c0 + hc * 16, dual, v);
#pragma unroll
            for (int i = 0; i < 16; ++i) acc_s[(hc * 16 + i) * 128 + f] = v[i];
        }
        epi_barrier(group);
        const int l4 = et & 31;
#pragma unroll
        for (int k = 0; k < kStagingCols / 4; ++k) {
            const int nl = (et >> 5) + 4 * k;
            if (c0 + nl < n_valid && l4 * 4 < feat_limit)
                *reinterpret_cast<float4*>(dst + (size_t)(c0 + nl) * row_stride + l4 * 4) =
                    *reinterpret_cast<const float4*>(acc_s + nl * 128 + l4 * 4);
        }
        epi_barrier(group);
    }
}

__device__ __forceinline__ int ld_acquire(const int* p) {
    int v;
    asm volatile("ld.acquire.gpu.global.s32 %0, [%1];" : "=r"(v) : "l"(p) : "memory");
    return v;
}
__device__ __forceinline__ void st_release(int* p, int v) {
    asm volatile("st.release.gpu.global.s32 [%0], %1;" ::"l"(p), "r"(v) : "memory");
}

// ---------------------------------------------------------------------------------------------------
// The kernel is written as its roles (W producer, X producer, two MMA issuers, epilogue warps), each a function over the
// CTA's share of one projection that carries its pipeline counters in and out.
// ---------------------------------------------------------------------------------------------------
struct CtaRange {
    int u0, u1;           // this CTA's units in the phase's unit space (see below; the unit count fits 32 bits, checked by the host)
    int vlen, koff;       // every tile owns vlen consecutive units, unit v of a tile being its K unit koff + v
    bool helper;
};

// The CTA's work is a range [u0, u1) of a unit space in which every tile owns vlen consecutive units.
//   split_s == 0, head_units == 0: all (tile, K) units, even contiguous shares ("stream-K"); vlen = n_ku.
//   split_s > 0: every tile cut into split_s aligned pieces.
//   head_units > 0: CTA t < n_tiles owns tile t and runs its first head_units K units; the CTAs after them
//     ("helpers") share the remaining units of all tiles evenly and only contribute partial tiles.
__device__ __forceinline__ CtaRange cta_range(const GemmDev& p, int cta) {
    CtaRange r;
    r.vlen = p.n_ku;
    r.koff = 0;
    r.helper = false;
    const int total = (int)p.total_units;
    if (p.head_units > 0) {
        if (cta < p.n_tiles) {
            r.vlen = p.head_units;
            r.u0 = cta * r.vlen;
            r.u1 = r.u0 + r.vlen;
        } else {
            r.helper = true;
            r.vlen = p.n_ku - p.head_units;
            r.koff = p.head_units;
            r.u0 = min(p.total_rem, (cta - p.n_tiles) * p.help_upc);
            r.u1 = min(p.total_rem, r.u0 + p.help_upc);
        }
    } else if (p.split_s > 0) {
        const int t0 = (cta / p.split_s) * p.n_ku;
        r.u0 = min(t0 + p.n_ku, t0 + (cta % p.split_s) * p.units_per_cta);
        r.u1 = min(t0 + p.n_ku, r.u0 + p.units_per_cta);
    } else {
        r.u0 = min(total, cta * p.units_per_cta);
        r.u1 = min(total, r.u0 + p.units_per_cta);
    }
    if (r.u1 < r.u0) r.u1 = r.u0;
    return r;
}

struct Pipe {               // the CTA's pipeline resources, the same for every phase of a launch
    uint8_t* stages;        // ring of S stages
    float* acc_s;           // [32][128] fp32 epilogue staging tile
    GemmCtrl* ctrl;
    volatile int* abort_flag;
    uint32_t tmem_acc;
    int S;
    int acc_stride;         // tensor-memory columns between the two accumulator buffers
    int dual;               // 1: every accumulator is two halves (columns +0 and +n_pad) summed by the epilogue
};

// One copy producer (a single thread): is_w streams W, else X.  A stage holds kUnitKb K blocks fetched by ONE copy of W
// (contiguous in the packed matrix) and ONE copy of X: a bulk copy costs its issuing thread a fixed ~0.45 us whatever
// its size (measured), so the two kinds of copies come from different threads.  i: units issued so far by this CTA
// over all phases (ring position).  Returns false after an abort.
__device__ __forceinline__ bool produce_units(const GemmDev& p, const CtaRange& r, const Pipe& pp, bool is_w, uint64_t pol, int& i) {
    // No division in the loop: the thread that issues the copies is the pace maker of the stream, and an integer
    // division costs it hundreds of cycles.  (tile, v): the unit's tile and its position among the tile's units;
    // (s, par): ring stage and the parity of the stage's "empty" phase to wait for.
    const int S = pp.S;
    const int n_units = r.u1 - r.u0;
    int tile = r.u0 / r.vlen, v = r.u0 - tile * r.vlen;
    int s = i % S;
    uint32_t par = ((uint32_t)(i / S) & 1u) ^ 1u;
    for (int k = 0; k < n_units; ++k, ++i) {
        if (i >= S && !mbar_wait(&pp.ctrl->empty[s], par, pp.abort_flag)) return false;
        const int kb = (r.koff + v) * kUnitKb;
        const int nk = min(kUnitKb, p.n_kb - kb);
        uint8_t* stage = pp.stages + (size_t)s * p.stage_bytes;
        if (is_w) {
            const uint32_t bytes = (uint32_t)nk * kWChunk;
            mbar_expect_tx(&pp.ctrl->full[s], bytes);
            bulk_load(stage, p.Wp + ((size_t)tile * p.n_kb + kb) * kWChunk, bytes, &pp.ctrl->full[s], pol);
            if (k == 0) GEMM_TL(2);
            if (k == n_units - 1) GEMM_TL(5);
        } else {
            const uint32_t bytes = (uint32_t)nk * p.x_chunk_bytes;
            mbar_expect_tx(&pp.ctrl->full[s], bytes);
            bulk_load(stage + kUnitKb * kWChunk, p.Xp + (size_t)kb * p.x_chunk_bytes, bytes, &pp.ctrl->full[s], pol);
            if (k == 0) GEMM_TL(11);
        }
        if (++s == S) { s = 0; par ^= 1u; }
        if (++v == r.vlen) { v = 0; ++tile; }
    }
    return true;
}

// After an abort: let the copies in flight land (bounded) before the CTA goes away.  i: units issued by this producer.
__device__ __forceinline__ void drain_after_abort(const Pipe& pp, int i) {
    volatile int ignore = 0;
    for (int j = max(0, i - pp.S); j < i; ++j) mbar_wait(&pp.ctrl->full[j % pp.S], (j / pp.S) & 1, &ignore);
}

// The MMA issuer (a single thread).  i: ring position, seg: accumulator segments so far (both over all phases).
__device__ __forceinline__ bool mma_units(const GemmDev& p, const CtaRange& r, const Pipe& pp, int& i, int& seg, int half) {
    const int S = pp.S;
    const uint32_t idesc = umma_idesc_bf16_m128(p.n_pad);
    const int k_lo = pp.dual ? 2 * half : 0, k_hi = pp.dual ? 2 * half + 2 : 4;
    bool ok = true;
    // as in produce_units: no division per unit.  v: position of unit u among its tile's units
    int u = r.u0, v = r.u0 % r.vlen;
    int s = i % S;
    uint32_t par = (uint32_t)(i / S) & 1u;
    while (u < r.u1 && ok) {
        const int seg_end = min(r.u1, u + (r.vlen - v));
        const int b = seg & 1;
        if (seg >= 2) ok = mbar_wait(&pp.ctrl->acc_empty[b], ((seg >> 1) - 1) & 1, pp.abort_flag);
        tc_fence_after_sync();
        const uint32_t d_addr = pp.tmem_acc + (uint32_t)(b * pp.acc_stride + half * p.n_pad);
        bool first = true;
        for (; u < seg_end && ok; ++u, ++i, ++v) {
            ok = mbar_wait(&pp.ctrl->full[s], par, pp.abort_flag);
            if (!ok) break;
            if (half == 0 && u == r.u0) GEMM_TL(3);
            if (half == 0 && u == r.u1 - 1) GEMM_TL(6);
            tc_fence_after_sync();
            const int kb = (r.koff + v) * kUnitKb;
            const int nk = min(kUnitKb, p.n_kb - kb);
            const uint32_t a_addr = smem_u32(pp.stages + (size_t)s * p.stage_bytes);
            const uint32_t b_addr = a_addr + kUnitKb * kWChunk;
            for (int j = 0; j < nk; ++j) {
                const uint64_t da = umma_desc_sw128(a_addr + j * kWChunk);
                const uint64_t db = umma_desc_sw128(b_addr + j * p.x_chunk_bytes);
                for (int k = k_lo; k < k_hi; ++k) umma_bf16(d_addr, da + 2 * k, db + 2 * k, idesc, !(first && k == k_lo));
                first = false;
            }
            umma_commit(&pp.ctrl->empty[s]);
            if (++s == S) { s = 0; par ^= 1u; }
        }
        if (v == r.vlen) v = 0;
        umma_commit(&pp.ctrl->acc_full[b]);   // also on abort, so that the epilogue warps wake up
        ++seg;
    }
    return ok;
}

// One group of four epilogue warps (128 threads) over the CTA's share of the projection.  seg: accumulator segments so far.
template <int EPI>
__device__ __forceinline__ void epilogue_units(const GemmDev& p, const CtaRange& r, const Pipe& pp, int cta, int warp, int lane,
                                               int group, int& seg, bool& ok) {
    // Two groups of four warps share every accumulator: group g takes the 32-node staging rounds g, g + 2, ... (trees of
    // up to 32 nodes leave group 1 nothing to do but arrive).  Each group has its own staging tile and its own barrier.
    const int q4 = warp & 3;               // TMEM lane quadrant this warp may read
    const int f = q4 * 32 + lane;          // accumulator row = weight row inside the tile
    const int ew = group == 0 ? warp - 2 : warp - 8;   // warp index inside the group
    const int et = ew * 32 + lane;         // 0..127 among the group's threads
    float* const acc_s = pp.acc_s + (size_t)group * kStagingCols * 128;
    const int c_first = group * kStagingCols, c_step = kEpiGroups * kStagingCols;
    for (int u = r.u0; u < r.u1; ++seg) {
        const int tile = u / r.vlen;
        const int tile_begin = tile * r.vlen;
        const int tile_end = tile_begin + r.vlen;
        const int seg_end = min(r.u1, tile_end);
        const bool tail = (seg_end == tile_end);
        const bool head = !r.helper && (u == tile_begin);
        u = seg_end;
        const int b = seg & 1;
        int head_cta = 0, last_cta = 0;         // stream-K: the CTAs that share this tile
        int g_first = 0, g_n = 0, my_slot = cta;   // contributors' slots this (owning) piece adds; slot a contributor writes
        if (p.head_units > 0) {
            // the tile's remaining units [tile * R, (tile + 1) * R) are spread over at most two helpers
            const int R = p.n_ku - p.head_units;
            const int j0 = (tile * R) / p.help_upc, j1 = ((tile + 1) * R - 1) / p.help_upc;
            g_first = 2 * tile;
            g_n = j1 - j0 + 1;
            if (r.helper) my_slot = 2 * tile + ((cta - p.n_tiles) - j0);
        } else {
            head_cta = tile_begin / p.units_per_cta;
            last_cta = (tile_end - 1) / p.units_per_cta;
            g_first = cta + 1;
            g_n = (head && !tail) ? last_cta - cta : 0;
        }
        // A tile this CTA owns but shares with other CTAs: their partial tiles are usually published long before
        // this CTA's own part is accumulated, so fetch them (the group's first 32 nodes) while waiting for the accumulator.
        const bool gather = head && g_n > 0 && EPI != EPI_PARTIAL;
        float pre[kStagingCols];
        if (ok && gather) {
            if (et == 0) {
                unsigned long long t0 = globaltimer_ns();
                for (int c2 = g_first; c2 < g_first + g_n; ++c2) {
                    while (ld_acquire(p.fix_flags + c2) == 0) {
                        if (*pp.abort_flag || globaltimer_ns() - t0 > g_wait_limit_ns) { *pp.abort_flag = 1; break; }
                    }
                }
            }
            epi_barrier(group);
            ok = !*pp.abort_flag;
#pragma unroll
            for (int cc = 0; cc < kStagingCols / 16; ++cc) {
#pragma unroll
                for (int i = 0; i < 16; ++i) pre[cc * 16 + i] = 0.f;
                if (ok && c_first + cc * 16 < p.n_pad) {
                    for (int c2 = g_first; c2 < g_first + g_n; ++c2) {
                        const float* src = p.fix_part + (size_t)c2 * p.n_pad * 128 + (size_t)(c_first + cc * 16) * 128 + f;
#pragma unroll
                        for (int i = 0; i < 16; ++i) pre[cc * 16 + i] += __ldcg(src + (size_t)i * 128);
                    }
                }
            }
        }
        int mat = 0, row0;
        if (EPI == EPI_SWIGLU) row0 = tile * 64;
        else { mat = tile / p.tiles_per_mat; row0 = (tile - mat * p.tiles_per_mat) * 128; }
        // EPI_QKV: a thread rotates 4 feature pairs (lo, lo + head_dim / 2) of every eighth node, so it needs the 4
        // (cos, sin) of each of its nodes once.  Those of the group's first staging round are fetched here, while the
        // accumulator is still being summed: their trip from L2 otherwise sits between the last MMA and the stores
        // (1.5 us per q/k tile, measured).
        constexpr int kRopeNodes = kStagingCols / 8;       // nodes per thread and staging round
        const int rope_half = p.head_dim >> 1;
        const int rope_pj = (et & 15) * 4;                  // first of the thread's 4 pairs among the tile's 64
        const int rope_hin = EPI == EPI_QKV ? rope_pj / rope_half : 0;          // head inside the tile
        const int rope_ri = rope_pj - rope_hin * rope_half;                     // rotary index of the first pair
        float4 cs0[kRopeNodes][2];
        if (EPI == EPI_QKV && ok && head && mat < 2) {
            const int n_hi0 = min(kStagingCols, p.T - c_first);
#pragma unroll
            for (int it = 0; it < kRopeNodes; ++it) {
                const int nl = (et >> 4) + 8 * it;
                const float4* src = reinterpret_cast<const float4*>(p.rope + (size_t)(c_first + nl) * rope_half + rope_ri);
                cs0[it][0] = nl < n_hi0 ? __ldg(src) : make_float4(1.f, 0.f, 1.f, 0.f);
                cs0[it][1] = nl < n_hi0 ? __ldg(src + 1) : make_float4(1.f, 0.f, 1.f, 0.f);
            }
        }
        if (ok) ok = mbar_wait(&pp.ctrl->acc_full[b], (seg >> 1) & 1, pp.abort_flag);
        ok = ok && !*pp.abort_flag;
        if (et == 0 && group == 0 && u >= r.u1) GEMM_TL(7);
        tc_fence_after_sync();
        const uint32_t taddr = pp.tmem_acc + ((uint32_t)(q4 * 32) << 16) + (uint32_t)(b * pp.acc_stride);
        const uint32_t dual = pp.dual ? (uint32_t)p.n_pad : 0u;

        if (!ok) {
            // nothing: fall through to the arrive below so that nobody waits on this accumulator
        } else if (EPI == EPI_PARTIAL) {
            const int feat = row0 + f;
            const int piece = p.split_s > 0 ? cta % p.split_s : cta - head_cta;
            store_tile_transposed(taddr, dual, p.n_pad, p.T, acc_s, f, et, group, p.part + (size_t)piece * p.part_stride + row0,
                                  (size_t)p.n_out, p.n_out - row0);
            if (group == 0 && head && p.split_s == 0 && feat < p.n_out) {   // slots no piece of this tile writes must read as zero
                for (int sl = last_cta - head_cta + 1; sl < p.max_pieces; ++sl) {
                    float* z = p.part + (size_t)sl * p.part_stride + feat;
                    for (int n = 0; n < p.T; ++n) z[(size_t)n * p.n_out] = 0.f;
                }
            }
        } else if (!head) {
            // a later piece of a tile another CTA owns: publish the raw fp32 partial tile
            store_tile_transposed(taddr, dual, p.n_pad, p.n_pad, acc_s, f, et, group, p.fix_part + (size_t)my_slot * p.n_pad * 128, 128, 128);
            epi_barrier_all();       // both groups have stored their rounds; the barrier orders those stores before the release below
            if (group == 0 && et == 0 && !p.dbg_skip_publish) {
                __threadfence();
                st_release(p.fix_flags + my_slot, 1);
            }
        } else {
            // this CTA owns the tile: add the other pieces (if any), then the fused epilogue
#pragma unroll
            for (int qi = 0; qi < CATS_MAX_TREE / kStagingCols / kEpiGroups; ++qi) {
                const int c0 = c_first + qi * c_step;
                if (c0 >= p.T || !ok) break;
#pragma unroll
                for (int hc = 0; hc < kStagingCols / 16; ++hc) {
                    const int c = hc * 16;
                    if (c0 + c >= p.n_pad) break;
                    float v[16];
                    acc_ld16(taddr + c0 + c, dual, v);
                    if (gather) {
                        if (qi == 0) {
#pragma unroll
                            for (int i = 0; i < 16; ++i) v[i] += pre[hc * 16 + i];
                        } else {
                            for (int c2 = g_first; c2 < g_first + g_n; ++c2) {
                                const float* src = p.fix_part + (size_t)c2 * p.n_pad * 128 + (size_t)(c0 + c) * 128 + f;
#pragma unroll
                                for (int i = 0; i < 16; ++i) v[i] += __ldcg(src + (size_t)i * 128);
                            }
                        }
                    }
                    if (EPI == EPI_LMHEAD && p.logits != nullptr && row0 + f < p.n_out) {
#pragma unroll
                        for (int i = 0; i < 16; ++i) {
                            int n = c0 + c + i;
                            if (n < p.T) p.logits[(size_t)n * p.n_out + row0 + f] = v[i];
                        }
                    }
#pragma unroll
                    for (int i = 0; i < 16; ++i) acc_s[(c + i) * 128 + f] = v[i];
                }
                epi_barrier(group);
                const int n_hi = min(kStagingCols, p.T - c0);   // valid nodes in this staging tile
                if (EPI == EPI_QKV) {
                    // thread -> 4 rotary pairs: features [lo, lo + 4) and [lo + half, lo + half + 4) of every eighth node,
                    // two 8-byte stores per node.  All loads of the thread are issued before the first store.
                    const int lo = rope_hin * p.head_dim + rope_ri, hi = lo + rope_half;
                    constexpr int NI = kRopeNodes;
                    if (row0 + hi < p.n_out) {
                        uint2 plo[NI], phi[NI];
                        if (mat < 2) {
                            float4 cs[NI][2];     // (cos, sin) of the 4 pairs
#pragma unroll
                            for (int it = 0; it < NI; ++it) {
                                const int nl = (et >> 4) + 8 * it;
                                const float4* src = reinterpret_cast<const float4*>(p.rope + (size_t)(c0 + nl) * rope_half + rope_ri);
#pragma unroll
                                for (int q = 0; q < 2; ++q) {
                                    if (qi == 0) cs[it][q] = cs0[it][q];       // fetched before the accumulator wait
                                    else cs[it][q] = nl < n_hi ? __ldg(src + q) : make_float4(1.f, 0.f, 1.f, 0.f);
                                }
                            }
#pragma unroll
                            for (int it = 0; it < NI; ++it) {
                                const int nl = (et >> 4) + 8 * it;
                                const float4 x = *reinterpret_cast<const float4*>(acc_s + nl * 128 + lo);
                                const float4 y = *reinterpret_cast<const float4*>(acc_s + nl * 128 + hi);
                                const float4 c0s = cs[it][0], c1s = cs[it][1];
                                plo[it].x = pack_bf16x2(x.x * c0s.x - y.x * c0s.y, x.y * c0s.z - y.y * c0s.w);
                                plo[it].y = pack_bf16x2(x.z * c1s.x - y.z * c1s.y, x.w * c1s.z - y.w * c1s.w);
                                phi[it].x = pack_bf16x2(y.x * c0s.x + x.x * c0s.y, y.y * c0s.z + x.y * c0s.w);
                                phi[it].y = pack_bf16x2(y.z * c1s.x + x.z * c1s.y, y.w * c1s.z + x.w * c1s.w);
                            }
                        } else {
#pragma unroll
                            for (int it = 0; it < NI; ++it) {
                                const int nl = (et >> 4) + 8 * it;
                                const float4 x = *reinterpret_cast<const float4*>(acc_s + nl * 128 + lo);
                                const float4 y = *reinterpret_cast<const float4*>(acc_s + nl * 128 + hi);
                                plo[it] = make_uint2(pack_bf16x2(x.x, x.y), pack_bf16x2(x.z, x.w));
                                phi[it] = make_uint2(pack_bf16x2(y.x, y.y), pack_bf16x2(y.z, y.w));
                            }
                        }
                        uint16_t* base;
                        if (mat == 0) base = p.q_out + (size_t)c0 * p.n_out;
                        else base = (mat == 1 ? p.kcache : p.vcache) + (size_t)(p.prefix_len + (p.kv_rows == nullptr ? c0 : 0)) * p.n_out;
#pragma unroll
                        for (int it = 0; it < NI; ++it) {
                            const int nl = (et >> 4) + 8 * it;
                            if (nl < n_hi) {
                                // a subset of the tree: row t of the batch is tree node kv_rows[t] (K and V only)
                                const size_t row = (mat == 0 || p.kv_rows == nullptr) ? (size_t)nl : (size_t)__ldg(p.kv_rows + c0 + nl);
                                uint16_t* dst = base + row * p.n_out + row0;
                                *reinterpret_cast<uint2*>(dst + lo) = plo[it];
                                *reinterpret_cast<uint2*>(dst + hi) = phi[it];
                            }
                        }
                    }
                } else if (EPI == EPI_SWIGLU) {
                    // features beyond n_out come out as silu(0)*0 = 0 (zero-padded weights): they are stored too,
                    // so that the padded K block of the down projection's input reads as zeros.
                    // thread -> 8 consecutive features = one 16-byte group of the packed layout, every 16th node
                    const int j8 = (et & 7) * 8;
                    const int feat = row0 + j8;
                    constexpr int NI = kStagingCols / 16;
#pragma unroll
                    for (int it = 0; it < NI; ++it) {
                        const int nl = (et >> 3) + 16 * it;
                        const float4 g0 = *reinterpret_cast<const float4*>(acc_s + nl * 128 + j8);
                        const float4 g1 = *reinterpret_cast<const float4*>(acc_s + nl * 128 + j8 + 4);
                        const float4 u0 = *reinterpret_cast<const float4*>(acc_s + nl * 128 + 64 + j8);
                        const float4 u1 = *reinterpret_cast<const float4*>(acc_s + nl * 128 + 64 + j8 + 4);
                        uint4 o;
                        o.x = pack_bf16x2(__fdividef(g0.x, 1.f + __expf(-g0.x)) * u0.x, __fdividef(g0.y, 1.f + __expf(-g0.y)) * u0.y);
                        o.y = pack_bf16x2(__fdividef(g0.z, 1.f + __expf(-g0.z)) * u0.z, __fdividef(g0.w, 1.f + __expf(-g0.w)) * u0.w);
                        o.z = pack_bf16x2(__fdividef(g1.x, 1.f + __expf(-g1.x)) * u1.x, __fdividef(g1.y, 1.f + __expf(-g1.y)) * u1.y);
                        o.w = pack_bf16x2(__fdividef(g1.z, 1.f + __expf(-g1.z)) * u1.z, __fdividef(g1.w, 1.f + __expf(-g1.w)) * u1.w);
                        if (nl < n_hi) *reinterpret_cast<uint4*>(p.act_out + packed_act_offset(c0 + nl, feat >> 3, p.n_pad)) = o;
                    }
                } else if (EPI == EPI_LMHEAD) {
                    for (int nl = ew; nl < n_hi; nl += 4) {
                        float best = -INFINITY;
                        int bi = 0x7fffffff;
#pragma unroll
                        for (int i = 0; i < 4; ++i) {
                            int ff = lane + 32 * i;
                            float v = acc_s[nl * 128 + ff];
                            if (row0 + ff < p.n_out && v > best) { best = v; bi = row0 + ff; }
                        }
#pragma unroll
                        for (int o = 16; o > 0; o >>= 1) {
                            float ov = __shfl_xor_sync(0xffffffffu, best, o);
                            int oi = __shfl_xor_sync(0xffffffffu, bi, o);
                            if (ov > best || (ov == best && oi < bi)) { best = ov; bi = oi; }
                        }
                        if (lane == 0) {
                            p.pmax[(size_t)tile * 128 + c0 + nl] = best;
                            p.pidx[(size_t)tile * 128 + c0 + nl] = bi;
                        }
                        if (p.psum != nullptr) {
                            // softmax statistics of this vocabulary tile at the given temperature, relative to the
                            // tile's own maximum: Z = sum e, S1 = sum e * (logit - max), e = exp((logit - max) / t)
                            float z = 0.f, s1 = 0.f;
#pragma unroll
                            for (int i = 0; i < 4; ++i) {
                                int ff = lane + 32 * i;
                                if (row0 + ff < p.n_out) {
                                    float d = acc_s[nl * 128 + ff] - best;
                                    float e = exp2f(d * p.inv_temp_log2e);
                                    z += e;
                                    s1 = fmaf(e, d, s1);
                                }
                            }
#pragma unroll
                            for (int o = 16; o > 0; o >>= 1) {
                                z += __shfl_xor_sync(0xffffffffu, z, o);
                                s1 += __shfl_xor_sync(0xffffffffu, s1, o);
                            }
                            if (lane == 0) {
                                p.psum[(size_t)tile * 128 + c0 + nl] = z;
                                p.ps1[(size_t)tile * 128 + c0 + nl] = s1;
                            }
                        }
                    }
                    if (p.cand != nullptr && et > 0 && et < p.T) {
                        // logit of tree node et's own token under its parent's distribution, if this tile holds it
                        const int pa = __ldg(p.tree_parent + et), tk = __ldg(p.tree_tokens + et);
                        if (pa >= c0 && pa < c0 + n_hi && tk >= row0 && tk < row0 + 128 && tk < p.n_out)
                            p.cand[et] = acc_s[(pa - c0) * 128 + (tk - row0)];
                    }
                }
                epi_barrier(group);
            }
            if (gather) {
                epi_barrier_all();       // both groups have seen the flags
                if (group == 0 && et == 0)
                    for (int c2 = g_first; c2 < g_first + g_n; ++c2) p.fix_flags[c2] = 0;   // leave the flags clear for the next launch
            }
        }
        tc_fence_before_sync();
        mbar_arrive(&pp.ctrl->acc_empty[b]);
        if (et == 0 && u >= r.u1) GEMM_TL(8 + group * 4);
    }
}

// Carves the dynamic shared memory, initialises the barriers and allocates tensor memory.  Every thread calls it.
// Returns false (after reporting) if the shared-memory window is not 1024-byte aligned; never seen violated.
__device__ __forceinline__ bool pipe_setup(Pipe& pp, uint8_t* smem_raw, int n_stages, uint32_t stage_bytes, uint32_t tmem_cols,
                                           int n_pad, int32_t* d_status) {
    pp.stages = smem_raw;                                                                   // 1024-byte aligned (checked)
    pp.acc_s = reinterpret_cast<float*>(pp.stages + (size_t)n_stages * stage_bytes);        // [kEpiGroups][32][128] fp32
    pp.ctrl = reinterpret_cast<GemmCtrl*>(reinterpret_cast<uint8_t*>(pp.acc_s) + kStagingBytes);
    pp.abort_flag = &pp.ctrl->abort_flag;
    pp.S = n_stages;
    pp.dual = kGemmDualIssue;
    pp.acc_stride = (kGemmDualIssue ? 2 : 1) * n_pad;
    if ((smem_u32(smem_raw) & 1023u) != 0) {   // the swizzled operand tiles need this alignment
        if (threadIdx.x == 0) report(d_status, CATS_ERR_UNSUPPORTED);
        return false;
    }
    GemmCtrl* ctrl = pp.ctrl;
    if (threadIdx.x == 0) {
        for (int s = 0; s < n_stages; ++s) {
            mbar_init(&ctrl->full[s], 2);      // one arrive.expect_tx from each copy producer
            mbar_init(&ctrl->empty[s], kGemmDualIssue ? 2 : 1);   // one commit from every MMA issuer
        }
        mbar_init(&ctrl->acc_full[0], kGemmDualIssue ? 2 : 1);
        mbar_init(&ctrl->acc_full[1], kGemmDualIssue ? 2 : 1);
        mbar_init(&ctrl->acc_empty[0], 128 * kEpiGroups);
        mbar_init(&ctrl->acc_empty[1], 128 * kEpiGroups);
        ctrl->abort_flag = 0;
        mbar_fence_init();
    }
    if ((threadIdx.x >> 5) == 1) {
        tmem_alloc(&ctrl->tmem_base, tmem_cols);
        tmem_relinquish();
    }
    tc_fence_before_sync();
    __syncthreads();
    tc_fence_after_sync();
    pp.tmem_acc = ctrl->tmem_base;
    return true;
}

__device__ __forceinline__ void pipe_teardown(const Pipe& pp, uint32_t tmem_cols, int32_t* d_status) {
    tc_fence_before_sync();
    __syncthreads();
    if ((threadIdx.x >> 5) == 1) {
        __syncwarp();
        tc_fence_after_sync();
        tmem_dealloc(pp.tmem_acc, tmem_cols);
    }
    if (threadIdx.x == 0 && pp.ctrl->abort_flag) report(d_status, CATS_ERR_TIMEOUT);
}

// Twelve warps: W producer, two MMA issuers, X producer, two groups of four epilogue warps.  Three warps share each of
// the SM's four register partitions (16 K registers), hence at most 170 registers per thread; all four epilogues fit
// without spilling.
#ifndef CATS_GEMM_MAXREG
#define CATS_GEMM_MAXREG 168      // 12 warps: three of them share one of the SM's four 16 K register partitions
#endif
template <int EPI>
__global__ void __maxnreg__(CATS_GEMM_MAXREG) k_gemm_sk(const GemmDev p) {
    extern __shared__ __align__(1024) uint8_t smem_raw[];
    Pipe pp;
#ifdef CATS_TIMELINE
    if (threadIdx.x == 0) {
        GEMM_TL(0);
        unsigned sm;
        asm volatile("mov.u32 %0, %%smid;" : "=r"(sm));
        p.tl[(size_t)blockIdx.x * kTlStamps + 10] = sm;
    }
#endif
    if (!pipe_setup(pp, smem_raw, p.n_stages, p.stage_bytes, p.tmem_cols, p.n_pad, p.d_status)) return;
    if (threadIdx.x == 0) GEMM_TL(1);
    pdl_launch_dependents();
    const int warp = threadIdx.x >> 5;
    const int lane = threadIdx.x & 31;
    const int cta = blockIdx.x;
    const CtaRange r = cta_range(p, cta);

    if (warp == 0 || warp == 6) {
        // ---------------- copy producers: warp 0 streams W, warp 6 streams X ----------------
        if (lane == 0) {
            const bool is_w = (warp == 0);
            const uint64_t pol = is_w ? l2_policy_evict_first() : l2_policy_evict_last();
            if (!is_w) {
                pdl_wait();    // activations come from the previous kernel; weights never do
                GEMM_TL(4);
            }
            int i = 0;
            produce_units(p, r, pp, is_w, pol, i);
            if (*pp.abort_flag) drain_after_abort(pp, i);
        }
    } else if (warp == 1) {
        // ---------------- MMA issuer ----------------
        if (lane == 0) {
            int i = 0, seg = 0;
            mma_units(p, r, pp, i, seg, 0);
        }
    } else if (warp == 7) {
        // ---------------- second MMA issuer: the other two K = 16 steps of every K block, into its own accumulator half ----------------
        if (kGemmDualIssue && lane == 0) {
            int i = 0, seg = 0;
            mma_units(p, r, pp, i, seg, 1);
        }
    } else {
        // ---------------- epilogue warps: group 0 = warps 2-5, group 1 = warps 8-11 ----------------
        pdl_wait();
        int seg = 0;
        bool ok = true;
        epilogue_units<EPI>(p, r, pp, cta, warp, lane, warp < 6 ? 0 : 1, seg, ok);
    }
    pipe_teardown(pp, p.tmem_cols, p.d_status);
    if (threadIdx.x == 0) GEMM_TL(9);
}

// ---------------------------------------------------------------------------------------------------
// Weight packing: nn.Linear [rows][cols] bf16 -> 16 KB chunks (tile, K block) in the tcgen05 K-major
// 128-byte-swizzle layout.  layout 0: n_src matrices stacked, each padded to whole 128-row tiles.
// layout 1: two matrices (gate, up) interleaved as tiles of 64 + 64 rows.  Rows and columns beyond
// the matrix are zero.  One thread per 16-byte group.
// ---------------------------------------------------------------------------------------------------
__global__ void __launch_bounds__(256) k_pack_weights(const uint16_t* __restrict__ s0, const uint16_t* __restrict__ s1,
                                                      const uint16_t* __restrict__ s2, int layout, int rows, int cols,
                                                      int tiles_per_mat, int n_kb, long long n_groups, uint4* __restrict__ dst) {
    long long g = (long long)blockIdx.x * blockDim.x + threadIdx.x;
    if (g >= n_groups) return;
    int c = (int)(g & 7);
    int r = (int)((g >> 3) & 127);
    long long chunk = g >> 10;
    int kb = (int)(chunk % n_kb);
    int tile = (int)(chunk / n_kb);
    const uint16_t* src;
    int row;
    if (layout == 1) {
        src = r < 64 ? s0 : s1;
        row = tile * 64 + (r & 63);
    } else {
        int mat = tile / tiles_per_mat;
        src = mat == 0 ? s0 : (mat == 1 ? s1 : s2);
        row = (tile - mat * tiles_per_mat) * 128 + r;
    }
    int col = kb * 64 + c * 8;
    uint4 v = make_uint4(0, 0, 0, 0);
    if (row < rows && col < cols) {
        if (col + 8 <= cols) {
            v = *reinterpret_cast<const uint4*>(src + (size_t)row * cols + col);
        } else {
            uint16_t tmp[8] = {0, 0, 0, 0, 0, 0, 0, 0};
            for (int i = 0; col + i < cols; ++i) tmp[i] = src[(size_t)row * cols + col + i];
            v = *reinterpret_cast<uint4*>(tmp);
        }
    }
    size_t off = (size_t)chunk * (kWChunk / 16) + (size_t)(r >> 3) * 64 + (size_t)(r & 7) * 8 + (size_t)(c ^ (r & 7));
    dst[off] = v;
}

size_t packed_weight_bytes(int n_src, int layout, int rows, int cols) {
    int n_kb = (cols + 63) / 64;
    long long tiles = layout == 1 ? (rows + 63) / 64 : (long long)n_src * ((rows + 127) / 128);
    return (size_t)tiles * n_kb * kWChunk;
}

cudaError_t launch_pack_weights(const void* const* src, int n_src, int layout, int rows, int cols, void* dst, cudaStream_t st) {
    int n_kb = (cols + 63) / 64;
    int tpm = (rows + 127) / 128;
    long long groups = (long long)(packed_weight_bytes(n_src, layout, rows, cols) / 16);
    long long blocks = (groups + 255) / 256;
    k_pack_weights<<<(unsigned)blocks, 256, 0, st>>>((const uint16_t*)src[0], (const uint16_t*)src[n_src > 1 ? 1 : 0],
                                                      (const uint16_t*)src[n_src > 2 ? 2 : 0], layout, rows, cols, tpm, n_kb, groups,
                                                      (uint4*)dst);
    ++g_launch_count;
    return cudaGetLastError();
}

// ---------------------------------------------------------------------------------------------------
// host side
// ---------------------------------------------------------------------------------------------------
// Time line of the projection launches (measurement builds): copies the stamps to the host, or clears them.
cudaError_t timeline_gemm(void* host, size_t bytes, bool clear) {
#ifdef CATS_TIMELINE
    if (clear) {
        void* b = nullptr;
        cudaError_t e = cudaGetSymbolAddress(&b, g_tl_gemm);
        g_tl_gemm_next = 0;
        return e != cudaSuccess ? e : cudaMemset(b, 0, sizeof(g_tl_gemm));
    }
    return cudaMemcpyFromSymbol(host, g_tl_gemm, bytes < sizeof(g_tl_gemm) ? bytes : sizeof(g_tl_gemm));
#else
    (void)host; (void)bytes; (void)clear;
    return cudaErrorNotSupported;
#endif
}

cudaError_t set_wait_limit_gemm(unsigned long long ns) { return cudaMemcpyToSymbol(g_wait_limit_ns, &ns, sizeof(ns)); }

int gemm_num_tiles(const GemmProblem& p) {
    if (p.epi == EPI_SWIGLU) return (p.n_out + 63) / 64;
    return p.n_mats * ((p.n_out + 127) / 128);
}

GemmPlan gemm_plan(const GemmProblem& p) {
    GemmPlan pl;
    const int n_ku = ((p.K + 63) / 64 + kUnitKb - 1) / kUnitKb;   // units (groups of kUnitKb K blocks) per tile
    const int tiles = gemm_num_tiles(p);
    const long long total = (long long)tiles * n_ku;
    long long upc = (total + kGemmCtas - 1) / kGemmCtas;          // stream-K: even, contiguous shares
    pl.head_units = 0;
    pl.help_upc = 0;
    if (p.epi == EPI_PARTIAL) {
        // partial sums: cut every tile into the same number of aligned pieces when that keeps most SMs busy (fewer
        // partial-sum slots for the following reduction, no zero filling), else even shares with a bounded number of
        // pieces.  (One whole tile per CTA for the fused epilogues was measured too: 96 SMs cannot pull what 148 can.)
        int s = kGemmCtas / tiles;
        if (s > kMaxPartSlots) s = kMaxPartSlots;
        if (s >= 2 && (long long)tiles * s * 10 >= kGemmCtas * 8 && n_ku >= s) {
            pl.split_s = s;
            pl.units_per_cta = (n_ku + s - 1) / s;
            pl.n_ctas = tiles * s;
            pl.max_pieces = s;
            return pl;
        }
        long long lim = (n_ku + kMaxPartSlots - 3) / (kMaxPartSlots - 2);
        if (upc < lim) upc = lim;
    }
    if (upc < 1) upc = 1;
    pl.head_units = 0;
    pl.help_upc = 0;
    if (p.epi != EPI_PARTIAL && upc < n_ku && tiles < kGemmCtas) {
        // Fewer tiles than CTAs and a fused epilogue.  With even shares some CTAs hold nothing but the middle of a tile:
        // they publish their partial tile only when the whole stream ends, and the tile's owner then still has to fetch
        // it and run its epilogue.  Instead: one owner CTA per tile runs the first `a` K units and the epilogue; the
        // other CTAs ("helpers") share the remaining units of all tiles, with shorter shares than an owner's, so their
        // partial tiles are in L2 before an owner needs them.  How much shorter grows with the tree (the published tiles
        // and the owner's epilogue grow with it).  Measured on the 7B forward (two MMA issuers), 32 units per tile, owner units a:
        //   T = 16:  a = 23 / 24 / 25 / 26 / 28 -> 2.926 / 2.896 / 2.889 / 2.906 / 2.937 ms
        //   T = 64:  a = 24 / 25 / 26 / 27 / 28 -> 3.322 / 3.301 / 3.230 / 3.241 / 3.255 ms
        //   T = 128: a = 25 / 26 / 27 / 28      -> 4.072 / 3.955 / 3.976 / 3.979 ms
        // (an owner's SM pulls more once the helpers have finished, so the optimum is flat towards large shares: with
        // a = 31, next to no help at all, the forward is only 2 % slower.)  Measured again with a quarter of the matrix on its
        // way into L2 when the kernel starts (lead = 7 / 8.5 / 10 / 11.5 / 13 units at T = 16, + 3 at T = 64, + 4.5 at T = 128):
        //   T = 16: 2.672 / 2.673 / 2.658 / 2.659 / 2.634 ms    T = 64: 2.840 / 2.848 / 2.796 / 2.794 / 2.794 ms
        //   T = 128: 3.50 / 3.46 / 3.41 / 3.45 / 3.47 ms  ->  13 units up to 64 nodes, 14.5 above.
        const int h = kGemmCtas - tiles;
        const double rho = (double)tiles / h;
        int lg = 0;                                    // log2(n_pad / 16): 0, 1, 2, 3 for trees of up to 16, 32, 64, 128 nodes
        for (int n = ((p.T + 15) / 16) * 16; n > 16; n = (n + 1) / 2) ++lg;
        const double lead = (lg <= 2 ? 13.0 : 10.0 + 1.5 * lg) * n_ku / 32.0;
        int a = (int)((rho * n_ku + lead) / (1.0 + rho) + 0.999);
        if (a > n_ku - 1) a = n_ku - 1;
        const int R = n_ku - a;
        if (a >= 1 && R >= 1) {
            const int hupc = (int)(((long long)tiles * R + h - 1) / h);
            if (hupc >= R) {           // a tile's remainder then meets at most two helpers (two slots per tile)
                pl.split_s = 0;
                pl.head_units = a;
                pl.help_upc = hupc;
                pl.units_per_cta = a;
                pl.n_ctas = tiles + (int)(((long long)tiles * R + hupc - 1) / hupc);
                pl.max_pieces = 1;
                return pl;
            }
        }
    }
    pl.split_s = 0;
    pl.units_per_cta = (int)upc;
    pl.n_ctas = (int)((total + upc - 1) / upc);
    // pieces of one tile: a range of n_ku units cut by boundaries every upc units
    pl.max_pieces = (n_ku % upc == 0) ? (int)(n_ku / upc) : (int)((n_ku + upc - 2) / upc) + 1;
    if (upc >= n_ku && upc % n_ku == 0) pl.max_pieces = 1;
    if (pl.max_pieces > kMaxPartSlots) pl.max_pieces = kMaxPartSlots;
    return pl;
}

namespace {
constexpr int kMaxSmem = 225 * 1024;   // leaves room for a co-resident RMSNorm CTA (see k_gemm_sk)

// Device-side description of one projection.  max_stages: upper bound on the ring depth (a single launch needs no more
// stages than a CTA has units).  Returns the dynamic shared memory the kernel needs.
size_t make_gemm_dev(const GemmProblem& p, const GemmPlan& pl, int max_stages, GemmDev& d) {
    d = GemmDev{};
    d.epi = p.epi;
    d.T = p.T;
    d.n_pad = ((p.T + 15) / 16) * 16;
    d.n_out = p.n_out;
    d.n_kb = (p.K + 63) / 64;
    d.n_ku = (d.n_kb + kUnitKb - 1) / kUnitKb;
    d.n_tiles = gemm_num_tiles(p);
    d.tiles_per_mat = (p.n_out + 127) / 128;
    d.total_units = (long long)d.n_tiles * d.n_ku;
    d.units_per_cta = pl.units_per_cta;
    d.max_pieces = pl.max_pieces;
    d.split_s = pl.split_s;
    d.head_units = pl.head_units;
    d.help_upc = pl.help_upc;
    d.total_rem = pl.head_units > 0 ? d.n_tiles * (d.n_ku - pl.head_units) : 0;
    d.x_chunk_bytes = (uint32_t)d.n_pad * 128;
    d.stage_bytes = kUnitKb * kWChunk + ((kUnitKb * d.x_chunk_bytes + 1023) / 1024) * 1024;
    int stages = (int)((kMaxSmem - kCtrlBytes - kStagingBytes) / d.stage_bytes);
    if (stages > kMaxStages) stages = kMaxStages;
    if (stages > max_stages) stages = max_stages;
    if (stages < 1) stages = 1;
    d.n_stages = stages;
    uint32_t cols = 32;
    while ((int)cols < (kGemmDualIssue ? 4 : 2) * d.n_pad) cols <<= 1;
    d.tmem_cols = cols;
    d.Wp = (const uint8_t*)p.W[0];
    d.Xp = (const uint8_t*)p.X;
    d.fix_part = p.fix_part;
    d.fix_flags = p.fix_flags;
    d.part = p.part;
    d.part_stride = p.part_stride;
    d.q_out = (uint16_t*)p.q_out;
    d.kcache = (uint16_t*)p.kcache;
    d.vcache = (uint16_t*)p.vcache;
    d.rope = p.rope;
    d.head_dim = p.head_dim;
    d.prefix_len = p.prefix_len;
    d.kv_rows = p.kv_rows;
    d.act_out = (uint8_t*)p.act_out;
    d.logits = p.logits;
    d.pmax = p.pmax;
    d.pidx = p.pidx;
    d.psum = p.psum;
    d.ps1 = p.ps1;
    d.inv_temp_log2e = p.inv_temperature * 1.4426950408889634f;
    d.tree_parent = p.tree_parent;
    d.tree_tokens = p.tree_tokens;
    d.cand = p.cand;
    d.d_status = p.d_status;
    d.dbg_skip_publish = g_debug_fault == 1 ? 1 : 0;
#ifdef CATS_TIMELINE
    {
        unsigned long long* base = nullptr;
        cudaGetSymbolAddress((void**)&base, g_tl_gemm);
        d.tl = base + (size_t)(g_tl_gemm_next++ % 512) * kTlCtas * kTlStamps;
    }
#endif
    return (size_t)stages * d.stage_bytes + kStagingBytes + kCtrlBytes;
}
}  // namespace

cudaError_t launch_gemm(const GemmProblem& p, cudaStream_t st) {
    static bool attr_set = false;
    if (!attr_set) {
        cudaError_t e = cudaFuncSetAttribute(k_gemm_sk<EPI_PARTIAL>, cudaFuncAttributeMaxDynamicSharedMemorySize, kMaxSmem);
        if (e == cudaSuccess) e = cudaFuncSetAttribute(k_gemm_sk<EPI_QKV>, cudaFuncAttributeMaxDynamicSharedMemorySize, kMaxSmem);
        if (e == cudaSuccess) e = cudaFuncSetAttribute(k_gemm_sk<EPI_SWIGLU>, cudaFuncAttributeMaxDynamicSharedMemorySize, kMaxSmem);
        if (e == cudaSuccess) e = cudaFuncSetAttribute(k_gemm_sk<EPI_LMHEAD>, cudaFuncAttributeMaxDynamicSharedMemorySize, kMaxSmem);
        if (e != cudaSuccess) return e;
        attr_set = true;
    }
    const GemmPlan pl = gemm_plan(p);
    GemmDev d;
    const size_t smem = make_gemm_dev(p, pl, pl.units_per_cta, d);
    if (d.total_units + (long long)kGemmCtas * pl.units_per_cta >= (1ll << 31)) return cudaErrorInvalidValue;   // the kernel counts units in 32 bits
    switch (p.epi) {
        case EPI_PARTIAL: return launch_pdl(k_gemm_sk<EPI_PARTIAL>, dim3(pl.n_ctas), dim3(kGemmThreads), smem, st, d);
        case EPI_QKV: return launch_pdl(k_gemm_sk<EPI_QKV>, dim3(pl.n_ctas), dim3(kGemmThreads), smem, st, d);
        case EPI_SWIGLU: return launch_pdl(k_gemm_sk<EPI_SWIGLU>, dim3(pl.n_ctas), dim3(kGemmThreads), smem, st, d);
        case EPI_LMHEAD: return launch_pdl(k_gemm_sk<EPI_LMHEAD>, dim3(pl.n_ctas), dim3(kGemmThreads), smem, st, d);
        default: return cudaErrorInvalidValue;
    }
}

}  // namespace cats
