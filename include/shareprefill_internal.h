/*
 * shareprefill_internal.h - exported hooks of the SharePrefill library that are
 * not part of its interface: kernel selection for A/B checks, the in-kernel phase
 * trace, and the launch counter.  Tests and the benchmark use them; applications
 * have no reason to.  The paper has no counterpart for any of them.
 */
#ifndef SHAREPREFILL_INTERNAL_H_
#define SHAREPREFILL_INTERNAL_H_

#include "shareprefill.h"

#ifdef __cplusplus
extern "C" {
#endif

/* Which attention kernel the context launches: 0 = tensor-core kernels
 * (tcgen05 / TMEM / TMA; the product path, default: for head_dim 128 and block
 * 128 the kernel that gives one CTA two adjacent row-blocks sharing their K/V
 * tiles, otherwise the one-row-block kernel), 1 = plain fp32 CUDA-core kernel
 * kept as an independent on-device cross-check, 2 = the one-row-block
 * tensor-core kernel for every shape, 3 = as 0, but every work item of the
 * paired kernel is two adjacent row-blocks of one head (0 also gives one item
 * to two heads of one KV head that walk the same list). */
int sp_ctx_set_kernel(sp_ctx* ctx, int which);

/* Phase trace of the tensor-core attention kernels (a profiling aid).  While a
 * buffer is set, the CTA that owns the longest row-block(s) of the first listed
 * head of every attention launch records, for each of its roles (0 = TMA
 * producer, 1 = MMA issuer (of the first row-block), 2 = softmax thread 0 of the
 * first row-block; paired kernel only: 3 = softmax thread 0 of the second
 * row-block, 4 = its MMA issuer), up to `events_per_role`
 * pairs {(event_id << 32) | step, SM clock} into
 * events[(role * events_per_role + n) * 2 .. +1].  Event ids: 20/21 K/V load
 * issued; 1 K tile landed, 2 QK^T issued, 3 P and V ready, 4 PV issued; 10 S
 * ready, 11 S in registers, 12 row max done, 13 exponentials done (paired
 * kernel: first half of P handed over), 14 O rescaled, 15 P stored and
 * signalled; paired kernel, issuer: 3/5 around the MMAs of the first
 * row-block, 6/4 around those of the second.  `events` is a device buffer of
 * 5 * events_per_role * 2 int64 that the caller zeroes; events_per_role = 0
 * switches tracing off. */
int sp_ctx_set_trace(sp_ctx* ctx, int64_t* events, int events_per_role);

/* Work order of a launch of the paired attention kernel (head_dim 128, block
 * 128), computed on the host exactly as the launcher does and walked exactly
 * as the kernel walks it: for every position raw = 0 .. n_heads *
 * ceil(n_row_blocks / 2) - 1 the two tiles of the work item,
 * tiles_out[4 raw ..] = {slot of tile A, row-block of tile A, slot of tile B,
 * row-block of tile B} (slots index `heads` / `lists`; a row-block >=
 * n_row_blocks means that the tile does not exist).  n_sm: SM count the launch
 * is sized for; pair_heads: as kernel selection 0 (non-zero) or 3 (zero).  Host
 * pointers; no device is touched.  For tests of the order. */
int sp_internal_pair_work_order(const int32_t* heads, const int32_t* lists, int n_heads, int n_q_heads, int n_kv_heads,
                                int n_row_blocks, int n_sm, int pair_heads, int32_t* tiles_out, int* n_groups_out);

/* Number of kernels this context has launched since creation (for callers
 * that account for launches). */
int64_t sp_ctx_launch_count(const sp_ctx* ctx);

#ifdef __cplusplus
}
#endif
#endif /* SHAREPREFILL_INTERNAL_H_ */
