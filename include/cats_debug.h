/*
 * cats_debug.h -- measurement and fault-injection hooks of libcats.
 *
 * These are not part of the product interface (include/cats.h): the benchmark
 * uses them to time parts of a forward, the tests use them to reach code that
 * normal operation never runs (the fallback attention kernel, the expiry of a
 * bounded device-side wait).  All state is process-wide, host-side except the
 * wait limit, and starts at the documented default.  None of them has a
 * counterpart in the paper.
 */
#ifndef CATS_DEBUG_H_
#define CATS_DEBUG_H_

#include "cats.h"

#ifdef __cplusplus
extern "C" {
#endif

/* Bit i of mask enables stage i of every decoder layer launched afterwards
 * (0 norm1, 1 qkv, 2 attention, 3 o-proj, 4 norm2, 5 gate/up, 6 down).
 * Default 0x7f: everything runs.  With stages disabled the results are
 * meaningless; only the timing of what still runs is of interest. */
void cats_debug_stage_mask(unsigned mask);

/* Byte offsets of the intermediate buffers inside the workspace
 * cats_workspace_bytes sizes: out[0..4] = xn, q, o, act (packed activation
 * layout, except q: [T][n_heads*head_dim] bf16) and part (fp32 split-K partial
 * sums [pieces][T][hidden]); out[5] = fp32 elements between two partial sums;
 * out[6], out[7] = pieces written by the O and the down projection.
 * out: HOST array of 8 size_t. */
int cats_debug_workspace_layout(const cats_model_cfg *cfg, int32_t T, size_t *out);

/* Attention kernel used for head_dim 128: -1 (default) chosen by shape, 0 the
 * mma.sync kernel (the fallback when the driver offers no tensor maps), 1 the
 * tcgen05 kernel, 2 the tcgen05 kernel with two softmax threads per query row
 * (by default every tree gets four). */
void cats_debug_attention_kernel(int which);

/* Limit of every bounded device-side wait, in nanoseconds, on the CURRENT
 * device (0 restores the default of 1 s).  Synchronises the device. */
int cats_debug_wait_limit_ns(unsigned long long ns);

/* Fault injection, host-made: launches issued afterwards withhold one signal
 * so that a bounded wait runs out (the kernel then reports CATS_ERR_TIMEOUT
 * through *d_status and returns; nothing traps, nothing waits without limit).
 *   0 none (default);
 *   1 projection kernel: CTAs that contribute a partial tile to a tile another
 *     CTA owns do not raise their ready flag;
 *   2 tcgen05 attention kernel: the loader announces the query tile on its
 *     barrier but never copies it.
 * Set a short wait limit first, or each expiry takes a second. */
void cats_debug_inject_fault(int which);

/* Measurement: which weights the kernels that leave HBM idle request into L2
 * for the projections after them.  which: 0 attention -> O projection,
 * 1 attention -> gate/up, 2 attention -> down, 3 the norm before QKV -> QKV,
 * 4 the norm before gate/up -> gate/up.  Of the matrix's 32 KB units every
 * period-th one is requested, starting at unit `phase`; period 0: none,
 * -1: the built-in choice (default for 1 and 3, the others default to 0).
 * Changes no result. */
void cats_debug_l2_warm(int which, int period, int phase);

/* Time line of the kernels inside a forward.  Only a library built with
 * -DCATS_TIMELINE records one (paper_2605_11186_b200/timeline.py builds it
 * beside the normal library and prints the table); the normal build returns
 * CATS_ERR_UNSUPPORTED.  kernel: 0 the projection kernel (512 launch slots),
 * 1 the tcgen05 attention kernel (128), 2 the register RMSNorm kernel (256);
 * a launch slot is [160 CTAs][16 stamps] of 64-bit %globaltimer values (ns),
 * zero where a CTA or stamp does not exist; the stamps are listed beside each
 * kernel in the sources.  host == NULL clears the slots and restarts the
 * numbering; else up to `bytes` bytes are copied to the HOST buffer. */
int cats_debug_timeline(int kernel, void *host, size_t bytes);

#ifdef __cplusplus
}
#endif
#endif /* CATS_DEBUG_H_ */
