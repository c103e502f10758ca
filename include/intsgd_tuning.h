/*
 * intsgd_tuning.h -- launch-shape knobs of the IntSGD step library.
 *
 * Not part of the stable interface of intsgd.h: these two calls exist for the library's own tests (every
 * kernel variant must give the same integers) and for timing experiments, and may change or disappear.
 * No result depends on them except the summation order of dx2.
 */
#ifndef INTSGD_TUNING_H_
#define INTSGD_TUNING_H_

#include "intsgd.h"

#ifdef __cplusplus
extern "C" {
#endif

/* Threads per block (multiple of 32, <= 512) and resident blocks per SM used to size the grids of the
 * direct (grid-stride) kernels.  0 keeps the built-in value. */
int intsgd_set_launch(intsgd_ctx* ctx, int32_t threads_per_block, int32_t blocks_per_sm);

/* Which kernels run the vector part of a step: 0 = automatic (the pipelined kernels -- bulk asynchronous
 * copies into a shared-memory ring -- when every pointer is 16-byte aligned and d <= 2^34, else the direct
 * kernels), 1 = always the direct kernels, 2 = same as 0.  Both give identical x, aggregate, payloads and
 * counters. */
int intsgd_set_fused_path(intsgd_ctx* ctx, int32_t path);

#ifdef __cplusplus
}
#endif
#endif /* INTSGD_TUNING_H_ */
