// Skinny weight-streaming GEMM for the projections of the tree-verification forward.
//
//   Y^T[n_out, T] = W[n_out, K] * X^T[K, T]        (W bf16 [n_out][K] as nn.Linear stores it,
//                                                    X bf16 [T][K], fp32 accumulation)
//
// The tree has at most 128 nodes, so the problem is bound by reading W once from HBM.  Each CTA owns
// one tile of 128 weight rows (the tcgen05 M dimension) and a range of K blocks; the T nodes, padded
// to a multiple of 16, are the N dimension.  Warp 0 streams W and X tiles through a ring of shared
// memory stages with TMA (128-byte swizzle), warp 1 issues tcgen05.mma into a TMEM accumulator, warps
// 2-5 read the accumulator back (tcgen05.ld) and run the fused epilogue:
//   EPI_PARTIAL  split-K partial sums (folded into the residual stream by the following RMSNorm kernel)
//   EPI_QKV      rotary embedding, bf16 q, k/v appended to the KV cache
//   EPI_SWIGLU   silu(gate) * up from a tile holding 64 gate rows and the matching 64 up rows
//   EPI_LMHEAD   fp32 logits and per-tile argmax candidates
// Weight tiles of the first stages are requested before griddepcontrol.wait: they do not depend on the
// previous kernel, so the stream keeps HBM busy across kernel boundaries.
// Every wait on an mbarrier is bounded; on expiry the CTA reports CATS_ERR_TIMEOUT, drains its copies
// in flight, frees its TMEM and returns.
#include "cats_kernels.cuh"

namespace cats {

int g_use_plain_gemm = 0;

struct GemmTmaps {
    CUtensorMap w[3];
    CUtensorMap x;
};

struct GemmDev {
    int epi, T, n_pad, K, n_out, n_mats, tiles_per_mat, n_kb, kb_per_split, n_stages;
    uint32_t stage_bytes, w_tile_bytes, x_tile_bytes, tmem_cols;
    float* part;
    size_t part_stride;
    uint16_t *q_out, *kcache, *vcache;
    const float2* rope;
    int head_dim, prefix_len;
    uint16_t* act_out;
    float* logits;
    float* pmax;
    int32_t* pidx;
    int32_t* d_status;
};

constexpr int kGemmThreads = 192;
constexpr int kCtrlBytes = 1024;
constexpr int kMaxStages = 12;

struct GemmCtrl {                 // lives in the first kCtrlBytes of dynamic shared memory
    uint64_t full[kMaxStages];
    uint64_t empty[kMaxStages];
    uint64_t accum;
    uint32_t tmem_base;
    int abort_flag;
};

__device__ __forceinline__ void epi_barrier() { asm volatile("bar.sync 1, 128;" ::: "memory"); }

__global__ void __launch_bounds__(kGemmThreads, 1) k_gemm_tc(const __grid_constant__ GemmTmaps tm, const GemmDev p) {
    extern __shared__ uint8_t smem_raw[];
    uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~(uintptr_t)1023);
    GemmCtrl* ctrl = reinterpret_cast<GemmCtrl*>(smem);
    uint8_t* stages = smem + kCtrlBytes;
    volatile int* abort_flag = &ctrl->abort_flag;

    const int warp = threadIdx.x >> 5;
    const int lane = threadIdx.x & 31;
    const int tile = blockIdx.x;
    const int split = blockIdx.y;
    const int kb0 = split * p.kb_per_split;
    const int kb1 = min(p.n_kb, kb0 + p.kb_per_split);
    const int nkb = max(0, kb1 - kb0);
    const int S = p.n_stages;

    // which weight matrix / row this tile covers
    int mat = 0, row0;
    if (p.epi == EPI_SWIGLU) {
        row0 = tile * 64;
    } else {
        mat = tile / p.tiles_per_mat;
        row0 = (tile - mat * p.tiles_per_mat) * 128;
    }

    if (threadIdx.x == 0) {
        for (int s = 0; s < S; ++s) {
            mbar_init(&ctrl->full[s], 1);
            mbar_init(&ctrl->empty[s], 1);
        }
        mbar_init(&ctrl->accum, 1);
        ctrl->abort_flag = 0;
        mbar_fence_init();
    }
    if (warp == 1) {
        tmem_alloc(&ctrl->tmem_base, p.tmem_cols);
        tmem_relinquish();
    }
    if (warp == 0 && lane == 0) {
        tma_prefetch_desc(&tm.w[0]);
        tma_prefetch_desc(&tm.x);
        if (p.n_mats > 1) tma_prefetch_desc(&tm.w[1]);
        if (p.n_mats > 2) tma_prefetch_desc(&tm.w[2]);
    }
    tc_fence_before_sync();
    __syncthreads();
    tc_fence_after_sync();
    pdl_launch_dependents();
    const uint32_t tmem_acc = ctrl->tmem_base;

    if (warp == 0) {
        // ---------------- TMA producer ----------------
        if (lane == 0) {
            const uint64_t pol_w = l2_policy_evict_first();
            const uint64_t pol_x = l2_policy_evict_last();
            auto issue_w = [&](int i) {
                int s = i % S;
                uint8_t* dst = stages + (size_t)s * p.stage_bytes;
                mbar_expect_tx(&ctrl->full[s], p.w_tile_bytes + p.x_tile_bytes);
                int x = (kb0 + i) * 64;
                if (p.epi == EPI_SWIGLU) {
                    tma_load_2d(dst, &tm.w[0], x, row0, &ctrl->full[s], pol_w);
                    tma_load_2d(dst + 8192, &tm.w[1], x, row0, &ctrl->full[s], pol_w);
                } else {
                    tma_load_2d(dst, &tm.w[mat], x, row0, &ctrl->full[s], pol_w);
                }
            };
            auto issue_x = [&](int i) {
                int s = i % S;
                uint8_t* dst = stages + (size_t)s * p.stage_bytes + p.w_tile_bytes;
                tma_load_2d(dst, &tm.x, (kb0 + i) * 64, 0, &ctrl->full[s], pol_x);
            };
            int pre = min(S, nkb);
            for (int i = 0; i < pre; ++i) issue_w(i);   // weights do not depend on the previous kernel
            pdl_wait();
            for (int i = 0; i < pre; ++i) issue_x(i);
            int issued = pre;
            for (int i = pre; i < nkb; ++i) {
                int s = i % S;
                if (!mbar_wait(&ctrl->empty[s], ((i / S) - 1) & 1, abort_flag)) break;
                issue_w(i);
                issue_x(i);
                issued = i + 1;
            }
            if (*abort_flag) {   // let the copies in flight land (bounded) before the CTA goes away
                volatile int ignore = 0;
                for (int i = max(0, issued - S); i < issued; ++i) mbar_wait(&ctrl->full[i % S], (i / S) & 1, &ignore);
            }
        }
    } else if (warp == 1) {
        // ---------------- MMA issuer ----------------
        if (lane == 0) {
            const uint32_t idesc = umma_idesc_bf16_m128(p.n_pad);
            for (int i = 0; i < nkb; ++i) {
                int s = i % S;
                if (!mbar_wait(&ctrl->full[s], (i / S) & 1, abort_flag)) break;
                tc_fence_after_sync();
                uint32_t a_addr = smem_u32(stages + (size_t)s * p.stage_bytes);
                uint64_t da = umma_desc_sw128(a_addr);
                uint64_t db = umma_desc_sw128(a_addr + p.w_tile_bytes);
#pragma unroll
                for (int k = 0; k < 4; ++k) umma_bf16(tmem_acc, da + 2 * k, db + 2 * k, idesc, (i | k) != 0);
                umma_commit(&ctrl->empty[s]);
            }
            umma_commit(&ctrl->accum);
        }
    } else {
        // ---------------- epilogue warps ----------------
        const int q4 = warp & 3;               // TMEM lane quadrant this warp may read
        const int f = q4 * 32 + lane;          // accumulator row = weight row inside the tile
        const int et = (warp - 2) * 32 + lane; // 0..127 thread index among the epilogue warps
        float* acc_s = reinterpret_cast<float*>(stages);   // [n][128] fp32, reuses the pipeline stages
        bool ok = true;
        if (nkb > 0) ok = mbar_wait(&ctrl->accum, 0, abort_flag);
        ok = ok && !*abort_flag;
        tc_fence_after_sync();
        pdl_wait();
        const int n_chunks = (p.T + 15) / 16;
        const uint32_t taddr = tmem_acc + ((uint32_t)(q4 * 32) << 16);
        if (ok) {
            if (p.epi == EPI_PARTIAL) {
                const int feat = row0 + f;
                float* dst = p.part + (size_t)split * p.part_stride + feat;
                for (int c = 0; c < n_chunks; ++c) {
                    float v[16];
                    if (nkb > 0) tmem_ld16(taddr + c * 16, v);
                    else {
#pragma unroll
                        for (int i = 0; i < 16; ++i) v[i] = 0.f;
                    }
                    if (feat < p.n_out) {
#pragma unroll
                        for (int i = 0; i < 16; ++i) {
                            int n = c * 16 + i;
                            if (n < p.T) dst[(size_t)n * p.n_out] = v[i];
                        }
                    }
                }
            } else {
                // stage the tile in shared memory so that threads can pair rows (RoPE halves, gate/up)
                for (int c = 0; c < n_chunks; ++c) {
                    float v[16];
                    tmem_ld16(taddr + c * 16, v);
                    if (p.epi == EPI_LMHEAD && p.logits != nullptr && row0 + f < p.n_out) {
#pragma unroll
                        for (int i = 0; i < 16; ++i) {
                            int n = c * 16 + i;
                            if (n < p.T) p.logits[(size_t)n * p.n_out + row0 + f] = v[i];
                        }
                    }
#pragma unroll
                    for (int i = 0; i < 16; ++i) acc_s[(c * 16 + i) * 128 + f] = v[i];
                }
            }
        }
        tc_fence_before_sync();
        if (p.epi != EPI_PARTIAL) {
            epi_barrier();
            if (ok && p.epi == EPI_QKV) {
                // thread -> feature pair (2j, 2j+1), every other node
                const int j2 = (et & 63) * 2;
                const int feat = row0 + j2;
                const int hd = p.head_dim, half = hd >> 1;
                const int in_head = feat % hd;
                const bool first_half = in_head < half;
                const int partner = first_half ? j2 + half : j2 - half;
                const int ri = in_head % half;
                if (feat < p.n_out) {
                    for (int n = et >> 6; n < p.T; n += 2) {
                        float x0 = acc_s[n * 128 + j2], x1 = acc_s[n * 128 + j2 + 1];
                        uint32_t packed;
                        if (mat < 2) {
                            float y0 = acc_s[n * 128 + partner], y1 = acc_s[n * 128 + partner + 1];
                            float2 cs0 = p.rope[(size_t)n * half + ri], cs1 = p.rope[(size_t)n * half + ri + 1];
                            float r0 = first_half ? x0 * cs0.x - y0 * cs0.y : x0 * cs0.x + y0 * cs0.y;
                            float r1 = first_half ? x1 * cs1.x - y1 * cs1.y : x1 * cs1.x + y1 * cs1.y;
                            packed = pack_bf16x2(r0, r1);
                        } else {
                            packed = pack_bf16x2(x0, x1);
                        }
                        uint16_t* base = mat == 0 ? p.q_out + (size_t)n * p.n_out
                                                  : (mat == 1 ? p.kcache : p.vcache) + (size_t)(p.prefix_len + n) * p.n_out;
                        *reinterpret_cast<uint32_t*>(base + feat) = packed;
                    }
                }
            } else if (ok && p.epi == EPI_SWIGLU) {
                const int j2 = (et & 31) * 2;
                const int feat = row0 + j2;
                if (feat < p.n_out) {
                    for (int n = et >> 5; n < p.T; n += 4) {
                        float g0 = acc_s[n * 128 + j2], g1 = acc_s[n * 128 + j2 + 1];
                        float u0 = acc_s[n * 128 + 64 + j2], u1 = acc_s[n * 128 + 64 + j2 + 1];
                        float a0 = g0 / (1.f + expf(-g0)) * u0;
                        float a1 = g1 / (1.f + expf(-g1)) * u1;
                        *reinterpret_cast<uint32_t*>(p.act_out + (size_t)n * p.n_out + feat) = pack_bf16x2(a0, a1);
                    }
                }
            } else if (ok && p.epi == EPI_LMHEAD) {
                for (int n = warp - 2; n < p.T; n += 4) {
                    float best = -INFINITY;
                    int bi = 0x7fffffff;
#pragma unroll
                    for (int i = 0; i < 4; ++i) {
                        int ff = lane + 32 * i;
                        float v = acc_s[n * 128 + ff];
                        if (row0 + ff < p.n_out && v > best) { best = v; bi = row0 + ff; }
                    }
#pragma unroll
                    for (int o = 16; o > 0; o >>= 1) {
                        float ov = __shfl_xor_sync(0xffffffffu, best, o);
                        int oi = __shfl_xor_sync(0xffffffffu, bi, o);
                        if (ov > best || (ov == best && oi < bi)) { best = ov; bi = oi; }
                    }
                    if (lane == 0) {
                        p.pmax[(size_t)tile * 128 + n] = best;
                        p.pidx[(size_t)tile * 128 + n] = bi;
                    }
                }
            }
        }
    }
    tc_fence_before_sync();
    __syncthreads();
    if (warp == 1) {
        __syncwarp();
        tc_fence_after_sync();
        tmem_dealloc(tmem_acc, p.tmem_cols);
    }
    if (threadIdx.x == 0 && ctrl->abort_flag) report(p.d_status, CATS_ERR_TIMEOUT);
}

// ---------------------------------------------------------------------------------------------------
// host side
// ---------------------------------------------------------------------------------------------------
typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*, const cuuint64_t*,
                                  const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave, CUtensorMapSwizzle,
                                  CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

static EncodeTiledFn get_encode_fn() {
    static EncodeTiledFn fn = nullptr;
    static bool tried = false;
    if (!tried) {
        tried = true;
        void* ptr = nullptr;
        cudaDriverEntryPointQueryResult qres;
        if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &ptr, cudaEnableDefault, &qres) == cudaSuccess &&
            qres == cudaDriverEntryPointSuccess)
            fn = reinterpret_cast<EncodeTiledFn>(ptr);
    }
    return fn;
}

// bf16 matrix [rows][cols] row-major, box of 64 columns x box_rows rows, 128-byte swizzle, zero fill
static bool encode_2d(CUtensorMap* tm, const void* base, int rows, int cols, int box_rows) {
    EncodeTiledFn fn = get_encode_fn();
    if (!fn) return false;
    cuuint64_t dims[2] = {(cuuint64_t)cols, (cuuint64_t)rows};
    cuuint64_t strides[1] = {(cuuint64_t)cols * 2};
    cuuint32_t box[2] = {64u, (cuuint32_t)box_rows};
    cuuint32_t estr[2] = {1u, 1u};
    CUresult r = fn(tm, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, const_cast<void*>(base), dims, strides, box, estr,
                    CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                    CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
    return r == CUDA_SUCCESS;
}

int gemm_num_tiles(const GemmProblem& p) {
    if (p.epi == EPI_SWIGLU) return (p.n_out + 63) / 64;
    return p.n_mats * ((p.n_out + 127) / 128);
}

cudaError_t launch_gemm(const GemmProblem& p, cudaStream_t st) {
    static bool attr_set = false;
    const int kMaxSmem = 227 * 1024;
    if (!attr_set) {
        cudaError_t e = cudaFuncSetAttribute(k_gemm_tc, cudaFuncAttributeMaxDynamicSharedMemorySize, kMaxSmem);
        if (e != cudaSuccess) return e;
        attr_set = true;
    }
    GemmTmaps tm;
    GemmDev d = {};
    d.epi = p.epi;
    d.T = p.T;
    d.n_pad = ((p.T + 15) / 16) * 16;
    d.K = p.K;
    d.n_out = p.n_out;
    d.n_mats = p.n_mats;
    d.tiles_per_mat = (p.n_out + 127) / 128;
    d.n_kb = (p.K + 63) / 64;
    int splits = p.epi == EPI_PARTIAL ? p.n_splits : 1;
    d.kb_per_split = (d.n_kb + splits - 1) / splits;
    if ((splits - 1) * d.kb_per_split >= d.n_kb && splits > 1) return cudaErrorInvalidValue;  // an empty split
    d.w_tile_bytes = 128 * 128;
    d.x_tile_bytes = (uint32_t)d.n_pad * 128;
    d.stage_bytes = d.w_tile_bytes + ((d.x_tile_bytes + 1023) / 1024) * 1024;
    int tiles = gemm_num_tiles(p);
    int ctas = tiles * splits;
    size_t budget = ctas <= 148 ? 200 * 1024 : 104 * 1024;
    int stages = (int)((budget - kCtrlBytes - 1024) / d.stage_bytes);
    if (stages > kMaxStages) stages = kMaxStages;
    if (stages > d.kb_per_split) stages = d.kb_per_split;
    if (stages < 2) stages = 2;
    size_t epi_bytes = p.epi == EPI_PARTIAL ? 0 : (size_t)d.n_pad * 128 * 4;
    size_t pipe_bytes = (size_t)stages * d.stage_bytes;
    size_t smem = 1024 + kCtrlBytes + (pipe_bytes > epi_bytes ? pipe_bytes : epi_bytes);
    if (smem > (size_t)kMaxSmem) return cudaErrorInvalidValue;
    d.n_stages = stages;
    uint32_t cols = 32;
    while ((int)cols < d.n_pad) cols <<= 1;
    d.tmem_cols = cols;
    d.part = p.part;
    d.part_stride = p.part_stride;
    d.q_out = (uint16_t*)p.q_out;
    d.kcache = (uint16_t*)p.kcache;
    d.vcache = (uint16_t*)p.vcache;
    d.rope = p.rope;
    d.head_dim = p.head_dim;
    d.prefix_len = p.prefix_len;
    d.act_out = (uint16_t*)p.act_out;
    d.logits = p.logits;
    d.pmax = p.pmax;
    d.pidx = p.pidx;
    d.d_status = p.d_status;

    int box_rows = p.epi == EPI_SWIGLU ? 64 : 128;
    for (int m = 0; m < 3; ++m) {
        const void* w = p.W[m < p.n_mats ? m : 0];
        if (!encode_2d(&tm.w[m], w, p.n_out, p.K, box_rows)) return cudaErrorUnknown;
    }
    if (!encode_2d(&tm.x, p.X, p.T, p.K, d.n_pad)) return cudaErrorUnknown;
    return launch_pdl(k_gemm_tc, dim3(tiles, splits), dim3(kGemmThreads), smem, st, tm, d);
}

// ---------------------------------------------------------------------------------------------------
// Plain CUDA-core version of the same problems (bring-up and cross-checks only; single split).
// scratch: fp32 [T][n_mats * n_out].
// ---------------------------------------------------------------------------------------------------
__global__ void __launch_bounds__(128) k_gemm_plain(const uint16_t* __restrict__ W, const uint16_t* __restrict__ X, int T,
                                                    int K, int n_out, float* __restrict__ Y, int ldy, int col0) {
    __shared__ float Ws[32][33];
    __shared__ float Xs[kMaxTree][33];
    pdl_wait();
    const int r = threadIdx.x & 31, g = threadIdx.x >> 5;
    const int row = blockIdx.x * 32 + r;
    float acc[32];
#pragma unroll
    for (int j = 0; j < 32; ++j) acc[j] = 0.f;
    for (int k0 = 0; k0 < K; k0 += 32) {
        for (int e = threadIdx.x; e < 32 * 32; e += 128) {
            int rr = e >> 5, kk = e & 31;
            int gr = blockIdx.x * 32 + rr;
            Ws[rr][kk] = (gr < n_out && k0 + kk < K) ? bf16_bits_to_float(W[(size_t)gr * K + k0 + kk]) : 0.f;
        }
        for (int e = threadIdx.x; e < T * 32; e += 128) {
            int t = e >> 5, kk = e & 31;
            Xs[t][kk] = (k0 + kk < K) ? bf16_bits_to_float(X[(size_t)t * K + k0 + kk]) : 0.f;
        }
        __syncthreads();
        for (int kk = 0; kk < 32; ++kk) {
            float w = Ws[r][kk];
#pragma unroll
            for (int j = 0; j < 32; ++j) {
                int t = g + 4 * j;
                if (t < T) acc[j] += w * Xs[t][kk];
            }
        }
        __syncthreads();
    }
    if (row < n_out) {
#pragma unroll
        for (int j = 0; j < 32; ++j) {
            int t = g + 4 * j;
            if (t < T) Y[(size_t)t * ldy + col0 + row] = acc[j];
        }
    }
}

__global__ void __launch_bounds__(256) k_plain_epilogue(const GemmDev p, const float* __restrict__ Y, int ldy) {
    pdl_wait();
    const int t = blockIdx.y;
    const int f = blockIdx.x * 256 + threadIdx.x;
    if (f >= p.n_out) return;
    const float* y = Y + (size_t)t * ldy;
    if (p.epi == EPI_PARTIAL) {
        p.part[(size_t)t * p.n_out + f] = y[f];
    } else if (p.epi == EPI_QKV) {
        const int hd = p.head_dim, half = hd >> 1;
        const int in_head = f % hd;
        const bool first = in_head < half;
        const int partner = first ? f + half : f - half;
        float2 cs = p.rope[(size_t)t * half + in_head % half];
        for (int mat = 0; mat < 2; ++mat) {
            float x = y[mat * p.n_out + f], xp = y[mat * p.n_out + partner];
            float r = first ? x * cs.x - xp * cs.y : x * cs.x + xp * cs.y;
            uint16_t b = float_to_bf16_bits(r);
            if (mat == 0) p.q_out[(size_t)t * p.n_out + f] = b;
            else p.kcache[(size_t)(p.prefix_len + t) * p.n_out + f] = b;
        }
        p.vcache[(size_t)(p.prefix_len + t) * p.n_out + f] = float_to_bf16_bits(y[2 * p.n_out + f]);
    } else if (p.epi == EPI_SWIGLU) {
        float g = y[f], u = y[p.n_out + f];
        p.act_out[(size_t)t * p.n_out + f] = float_to_bf16_bits(g / (1.f + expf(-g)) * u);
    } else if (p.epi == EPI_LMHEAD) {
        if (p.logits) p.logits[(size_t)t * p.n_out + f] = y[f];
    }
}

__global__ void __launch_bounds__(128) k_plain_tile_argmax(const float* __restrict__ Y, int ldy, int T, int n_out,
                                                           float* __restrict__ pmax, int32_t* __restrict__ pidx) {
    pdl_wait();
    int t = threadIdx.x;
    if (t >= T) return;
    int tile = blockIdx.x;
    float best = -INFINITY;
    int bi = 0x7fffffff;
    for (int ff = 0; ff < 128; ++ff) {
        int f = tile * 128 + ff;
        if (f < n_out) {
            float v = Y[(size_t)t * ldy + f];
            if (v > best) { best = v; bi = f; }
        }
    }
    pmax[(size_t)tile * 128 + t] = best;
    pidx[(size_t)tile * 128 + t] = bi;
}

cudaError_t launch_gemm_plain(const GemmProblem& p, float* scratch, cudaStream_t st) {
    int ldy = p.n_mats * p.n_out;
    cudaError_t e = cudaSuccess;
    for (int m = 0; m < p.n_mats && e == cudaSuccess; ++m)
        e = launch_pdl(k_gemm_plain, dim3((p.n_out + 31) / 32), dim3(128), 0, st, (const uint16_t*)p.W[m],
                       (const uint16_t*)p.X, p.T, p.K, p.n_out, scratch, ldy, m * p.n_out);
    if (e != cudaSuccess) return e;
    GemmDev d = {};
    d.epi = p.epi; d.T = p.T; d.K = p.K; d.n_out = p.n_out; d.n_mats = p.n_mats;
    d.part = p.part; d.part_stride = p.part_stride;
    d.q_out = (uint16_t*)p.q_out; d.kcache = (uint16_t*)p.kcache; d.vcache = (uint16_t*)p.vcache;
    d.rope = p.rope; d.head_dim = p.head_dim; d.prefix_len = p.prefix_len;
    d.act_out = (uint16_t*)p.act_out; d.logits = p.logits; d.pmax = p.pmax; d.pidx = p.pidx; d.d_status = p.d_status;
    e = launch_pdl(k_plain_epilogue, dim3((p.n_out + 255) / 256, p.T), dim3(256), 0, st, d, (const float*)scratch, ldy);
    if (e != cudaSuccess) return e;
    if (p.epi == EPI_LMHEAD)
        e = launch_pdl(k_plain_tile_argmax, dim3((p.n_out + 127) / 128), dim3(128), 0, st, (const float*)scratch, ldy, p.T,
                       p.n_out, p.pmax, p.pidx);
    return e;
}

}  // namespace cats
