// Shared device helpers of libcats: status reporting, bf16 packing, and thin wrappers over the
// sm_100a PTX used by the kernels (mbarrier, TMA, tcgen05, programmatic dependent launch).
#pragma once

#include <cuda_bf16.h>
#include <cuda_runtime.h>
#include <stdint.h>

#include "../../include/cats.h"

namespace cats {

constexpr int kMaxTree = CATS_MAX_TREE;
constexpr unsigned long long kWaitLimitNs = 1000000000ull;  // every device-side wait gives up after 1 s
// The limit the waits of this translation unit actually use (one copy per .cu file, each with a host-side setter that
// the fault-injection hook cats_debug_wait_limit_ns calls); read on the slow path of a wait only.
static __device__ unsigned long long g_wait_limit_ns = kWaitLimitNs;

__device__ __forceinline__ void report(int32_t* d_status, int code) {
    if (d_status) atomicMin(d_status, code);
}

__device__ __forceinline__ unsigned long long globaltimer_ns() {
    unsigned long long t;
    asm volatile("mov.u64 %0, %%globaltimer;" : "=l"(t));
    return t;
}

__device__ __forceinline__ uint32_t smem_u32(const void* p) {
    return static_cast<uint32_t>(__cvta_generic_to_shared(p));
}

__device__ __forceinline__ float bf16_bits_to_float(uint16_t b) { return __uint_as_float(((uint32_t)b) << 16); }

__device__ __forceinline__ uint16_t float_to_bf16_bits(float f) {
    __nv_bfloat16 h = __float2bfloat16_rn(f);
    return *reinterpret_cast<uint16_t*>(&h);
}

__device__ __forceinline__ uint32_t pack_bf16x2(float lo, float hi) {
    return (uint32_t)float_to_bf16_bits(lo) | ((uint32_t)float_to_bf16_bits(hi) << 16);
}

// Byte offset of the 16-byte group holding elements k8*8 .. k8*8+7 of row t inside a packed activation
// buffer: one chunk of n_pad rows x 64 columns per K block, rows of 128 bytes with the 128-byte swizzle
// (the shared-memory layout tcgen05.mma reads).  Every producer of a GEMM input writes this layout.
__host__ __device__ __forceinline__ size_t packed_act_offset(int t, int k8, int n_pad) {
    int kb = k8 >> 3, c = k8 & 7;
    return (size_t)kb * n_pad * 128 + (size_t)(t >> 3) * 1024 + (size_t)(t & 7) * 128 + (size_t)((c ^ (t & 7)) << 4);
}

// ---- programmatic dependent launch ------------------------------------------------------------
// wait: blocks until every kernel this launch depends on has completed and its writes are visible.
__device__ __forceinline__ void pdl_wait() { asm volatile("griddepcontrol.wait;" ::: "memory"); }
// launch_dependents: lets the next kernel in the stream start its prologue.
__device__ __forceinline__ void pdl_launch_dependents() { asm volatile("griddepcontrol.launch_dependents;" ::: "memory"); }

// ---- time line (measurement builds only: -DCATS_TIMELINE) ---------------------------------------
// Every launch of the projection, attention and norm kernels gets a slot of [kTlCtas][kTlStamps] 64-bit words; a CTA's
// role threads store %globaltimer there at the points named in timeline.py.  Nothing of this exists in a normal build.
constexpr int kTlCtas = 160, kTlStamps = 16;
#ifdef CATS_TIMELINE
#define CATS_TL(base, slot) do { (base)[(size_t)(blockIdx.y * gridDim.x + blockIdx.x) * kTlStamps + (slot)] = globaltimer_ns(); } while (0)
#else
#define CATS_TL(base, slot) do { } while (0)
#endif

// ---- requests into L2 ----------------------------------------------------------------------------
// Weights a later kernel will stream, requested into L2 by a kernel that leaves HBM idle: of the 32 KB units of
// [ptr, ptr + bytes) every period-th one starting at unit `phase`, so that the later kernel draws on L2 and HBM at once.
struct WarmReq {
    const uint8_t* ptr;
    unsigned long long bytes;     // 0: nothing
    int period, phase;
};
constexpr unsigned kWarmUnit = 32768;
// Called by n_workers threads (me: the caller's index among them), best one per warp: a request costs its thread
// 60-120 ns and the lanes of a warp take turns.  The selected units are dealt out round robin, at most max_each per
// caller (what does not fit is simply not requested).
__device__ __forceinline__ void l2_warm(const WarmReq& w, unsigned me, unsigned n_workers, int max_each) {
    if (w.bytes == 0) return;
    const unsigned n_units = (unsigned)(w.bytes / kWarmUnit);
    int n = 0;
    for (unsigned u = (unsigned)w.phase + me * (unsigned)w.period; u < n_units && n < max_each; u += n_workers * (unsigned)w.period, ++n)
        asm volatile("cp.async.bulk.prefetch.L2.global [%0], %1;" ::"l"(w.ptr + (size_t)u * kWarmUnit), "r"(kWarmUnit) : "memory");
}
inline WarmReq warm_req(const void* ptr, size_t bytes, int period, int phase) {
    WarmReq w;
    const bool on = ptr != nullptr && period >= 1 && phase >= 0 && bytes >= kWarmUnit;
    w.ptr = on ? (const uint8_t*)ptr : nullptr;
    w.bytes = on ? (unsigned long long)bytes : 0ull;
    w.period = on ? period : 1;
    w.phase = on ? phase : 0;
    return w;
}

// ---- mbarrier -----------------------------------------------------------------------------------
__device__ __forceinline__ void mbar_init(uint64_t* bar, uint32_t count) {
    asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(smem_u32(bar)), "r"(count) : "memory");
}
__device__ __forceinline__ void mbar_fence_init() { asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory"); }
__device__ __forceinline__ void mbar_expect_tx(uint64_t* bar, uint32_t bytes) {
    asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(smem_u32(bar)), "r"(bytes) : "memory");
}
__device__ __forceinline__ void mbar_arrive(uint64_t* bar) {
    asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(smem_u32(bar)) : "memory");
}
__device__ __forceinline__ bool mbar_try_wait(uint64_t* bar, uint32_t parity) {
    uint32_t ok;
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\t"
        "selp.u32 %0, 1, 0, p;\n\t}"
        : "=r"(ok)
        : "r"(smem_u32(bar)), "r"(parity)
        : "memory");
    return ok != 0;
}
// Bounded wait.  Returns false if the phase did not complete within the limit or another thread of
// the CTA raised *abort_flag; the caller must then stop using the pipeline.
__device__ __forceinline__ bool mbar_wait(uint64_t* bar, uint32_t parity, volatile int* abort_flag) {
    if (mbar_try_wait(bar, parity)) return true;
    unsigned long long t0 = globaltimer_ns();
    for (uint32_t it = 1;; ++it) {
        if (mbar_try_wait(bar, parity)) return true;
        if ((it & 63u) == 0) {
            if (*abort_flag) return false;
            if (globaltimer_ns() - t0 > g_wait_limit_ns) {
                *abort_flag = 1;
                return false;
            }
        }
    }
}

// ---- TMA ----------------------------------------------------------------------------------------
__device__ __forceinline__ void tma_prefetch_desc(const void* tmap) {
    asm volatile("prefetch.tensormap [%0];" ::"l"(reinterpret_cast<uint64_t>(tmap)) : "memory");
}
__device__ __forceinline__ uint64_t l2_policy_evict_first() {
    uint64_t p;
    asm volatile("createpolicy.fractional.L2::evict_first.b64 %0, 1.0;" : "=l"(p));
    return p;
}
__device__ __forceinline__ uint64_t l2_policy_evict_last() {
    uint64_t p;
    asm volatile("createpolicy.fractional.L2::evict_last.b64 %0, 1.0;" : "=l"(p));
    return p;
}
// 2-D tiled load global -> shared, completion counted in bytes on an mbarrier.  x is the innermost
// coordinate (elements); x * element size must be a multiple of 16 bytes.
__device__ __forceinline__ void tma_load_2d(void* smem_dst, const void* tmap, int32_t x, int32_t y, uint64_t* bar,
                                            uint64_t policy) {
    asm volatile(
        "cp.async.bulk.tensor.2d.shared::cluster.global.mbarrier::complete_tx::bytes.L2::cache_hint"
        " [%0], [%1, {%2, %3}], [%4], %5;"
        ::"r"(smem_u32(smem_dst)), "l"(reinterpret_cast<uint64_t>(tmap)), "r"(x), "r"(y), "r"(smem_u32(bar)), "l"(policy)
        : "memory");
}

// ---- tcgen05 (5th-generation tensor cores, accumulators in tensor memory) -------------------------
__device__ __forceinline__ void tmem_alloc(uint32_t* smem_slot, uint32_t ncols) {  // whole warp
    asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(smem_slot)), "r"(ncols)
                 : "memory");
}
__device__ __forceinline__ void tmem_relinquish() {  // whole warp
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
}
__device__ __forceinline__ void tmem_dealloc(uint32_t taddr, uint32_t ncols) {  // whole warp
    asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(taddr), "r"(ncols) : "memory");
}
__device__ __forceinline__ void tc_fence_before_sync() { asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void tc_fence_after_sync() { asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory"); }

// Shared-memory matrix descriptor for a K-major bf16 tile stored as rows of 128 bytes with the
// 128-byte swizzle (what a TMA box of 64 bf16 columns with SWIZZLE_128B writes): groups of 8 rows
// are 1024 bytes apart.  The tile base must be 1024-byte aligned; advancing along K by 16 elements
// adds 32 bytes to the start address.
__device__ __forceinline__ uint64_t umma_desc_sw128(uint32_t smem_addr) {
    uint64_t d = 0;
    d |= (uint64_t)((smem_addr & 0x3FFFFu) >> 4);         // start address, 16-byte units
    d |= (uint64_t)1 << 16;                               // leading byte offset (unused with swizzle)
    d |= (uint64_t)(1024 >> 4) << 32;                     // stride byte offset between 8-row groups
    d |= (uint64_t)1 << 46;                               // descriptor version (sm_100)
    d |= (uint64_t)2 << 61;                               // SWIZZLE_128B
    return d;
}
// Instruction descriptor: D fp32, A and B bf16, both K-major, M = 128, N = n (multiple of 16).
__host__ __device__ __forceinline__ uint32_t umma_idesc_bf16_m128(int n) {
    return (1u << 4) | (1u << 7) | (1u << 10) | ((uint32_t)(n >> 3) << 17) | ((uint32_t)(128 >> 4) << 24);
}
// D[tmem] (+)= A[smem] * B[smem]; one thread issues for the CTA.
__device__ __forceinline__ void umma_bf16(uint32_t tmem_d, uint64_t desc_a, uint64_t desc_b, uint32_t idesc, bool accumulate) {
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "setp.ne.b32 p, %4, 0;\n\t"
        "tcgen05.mma.cta_group::1.kind::f16 [%0], %1, %2, %3, p;\n\t}"
        ::"r"(tmem_d), "l"(desc_a), "l"(desc_b), "r"(idesc), "r"((uint32_t)accumulate)
        : "memory");
}
// Arrives on the mbarrier once every MMA issued so far by this thread has completed.
__device__ __forceinline__ void umma_commit(uint64_t* bar) {
    asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(smem_u32(bar)) : "memory");
}
// Each thread of the warp reads 16 consecutive fp32 columns of its own TMEM lane.
__device__ __forceinline__ void tmem_ld16(uint32_t taddr, float* v) {
    uint32_t r[16];
    asm volatile(
        "tcgen05.ld.sync.aligned.32x32b.x16.b32 {%0, %1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15}, [%16];\n\t"
        "tcgen05.wait::ld.sync.aligned;"
        : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7]), "=r"(r[8]),
          "=r"(r[9]), "=r"(r[10]), "=r"(r[11]), "=r"(r[12]), "=r"(r[13]), "=r"(r[14]), "=r"(r[15])
        : "r"(taddr)
        : "memory");
#pragma unroll
    for (int i = 0; i < 16; ++i) v[i] = __uint_as_float(r[i]);
}

// Shared-memory matrix descriptor for an MN-major bf16 operand with the 128-byte swizzle: rows of 128 bytes hold 64
// consecutive elements of the M (or N) dimension for one K index; 8 such rows (K = 8) form a 1024-byte group, the
// groups of one 64-element block follow each other along K, and the next 64-element block starts lbo_bytes later.
// The base must be 1024-byte aligned; advancing along K by 16 adds 2048 bytes to the start address.
__device__ __forceinline__ uint64_t umma_desc_sw128_mn(uint32_t smem_addr, uint32_t lbo_bytes) {
    uint64_t d = 0;
    d |= (uint64_t)((smem_addr & 0x3FFFFu) >> 4);         // start address, 16-byte units
    d |= (uint64_t)((lbo_bytes >> 4) & 0x3FFFu) << 16;    // leading byte offset: between 64-element blocks
    d |= (uint64_t)(1024 >> 4) << 32;                     // stride byte offset: between groups of 8 K rows
    d |= (uint64_t)1 << 46;                               // descriptor version (sm_100)
    d |= (uint64_t)2 << 61;                               // SWIZZLE_128B
    return d;
}
// Instruction descriptor as above with B MN-major (bit 16).
__host__ __device__ __forceinline__ uint32_t umma_idesc_bf16_m128_bmn(int n) { return umma_idesc_bf16_m128(n) | (1u << 16); }
// D[tmem] (+)= A[tmem] * B[smem]: A is read from tensor memory (row = lane, two bf16 per 32-bit column, K-major).
__device__ __forceinline__ void umma_bf16_ts(uint32_t tmem_d, uint32_t tmem_a, uint64_t desc_b, uint32_t idesc, bool accumulate) {
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "setp.ne.b32 p, %4, 0;\n\t"
        "tcgen05.mma.cta_group::1.kind::f16 [%0], [%1], %2, %3, p;\n\t}"
        ::"r"(tmem_d), "r"(tmem_a), "l"(desc_b), "r"(idesc), "r"((uint32_t)accumulate)
        : "memory");
}
// Each thread of the warp writes 8 / 16 consecutive 32-bit columns of its own TMEM lane (no wait: see tmem_wait_st).
__device__ __forceinline__ void tmem_st8(uint32_t taddr, const uint32_t* r) {
    asm volatile("tcgen05.st.sync.aligned.32x32b.x8.b32 [%0], {%1, %2, %3, %4, %5, %6, %7, %8};"
                 ::"r"(taddr), "r"(r[0]), "r"(r[1]), "r"(r[2]), "r"(r[3]), "r"(r[4]), "r"(r[5]), "r"(r[6]), "r"(r[7])
                 : "memory");
}
__device__ __forceinline__ void tmem_st16(uint32_t taddr, const float* v) {
    asm volatile(
        "tcgen05.st.sync.aligned.32x32b.x16.b32 [%0], {%1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15, %16};"
        ::"r"(taddr), "r"(__float_as_uint(v[0])), "r"(__float_as_uint(v[1])), "r"(__float_as_uint(v[2])), "r"(__float_as_uint(v[3])),
          "r"(__float_as_uint(v[4])), "r"(__float_as_uint(v[5])), "r"(__float_as_uint(v[6])), "r"(__float_as_uint(v[7])),
          "r"(__float_as_uint(v[8])), "r"(__float_as_uint(v[9])), "r"(__float_as_uint(v[10])), "r"(__float_as_uint(v[11])),
          "r"(__float_as_uint(v[12])), "r"(__float_as_uint(v[13])), "r"(__float_as_uint(v[14])), "r"(__float_as_uint(v[15]))
        : "memory");
}
__device__ __forceinline__ void tmem_wait_st() { asm volatile("tcgen05.wait::st.sync.aligned;" ::: "memory"); }

}  // namespace cats
