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

/* Number of kernels this context has launched since creation (for callers
 * that account for launches). */
int64_t sp_ctx_launch_count(const sp_ctx* ctx);

#ifdef __cplusplus
}
#endif
#endif /* SHAREPREFILL_INTERNAL_H_ */
