/*
 * libdab measurement aid, kept apart from the method's entry points (include/dab.h).
 */
#ifndef DAB_PROBE_H
#define DAB_PROBE_H

#include <stdint.h>

#include "dab.h"

#ifdef __cplusplus
extern "C" {
#endif

/*
 * dab_popc_probe — not part of the method (the paper only says that binary dot products are counted with
 * population-count instructions, Section 4.2): runs `iters` rounds of independent AND + population-count + add
 * chains in every thread of a grid of `blocks` x 256 threads and writes one word per thread to d_sink
 * (blocks*256 words, device memory owned by the caller), so that a caller timing it obtains the device's
 * achievable rate for the inner operation of the population-count contraction kernel.
 * Word operations executed = blocks * 256 * iters * 16.  Returns DAB_ERR_INVALID_ARG for a null sink, blocks < 1
 * or iters < 0.
 */
dab_status dab_popc_probe(uint32_t* d_sink, int32_t blocks, int32_t iters, void* stream);

#ifdef __cplusplus
}
#endif
#endif
