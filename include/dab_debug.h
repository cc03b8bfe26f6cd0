/*
 * libdab checking aid, kept apart from the method's entry points (include/dab.h).  The paper has no
 * counterpart: this is the library's own stand-in for a memory checker.
 *
 * A library built with -DDAB_DEBUG_BOUNDS (python -m paper_1804_02941_b200.build --debug-bounds, which
 * writes libdab_debug.so beside libdab.so) compares every global-memory index its hot-path kernels form
 * (row and patch coders, packing, both contraction kernels) with the extent of the array it addresses.  A
 * violating store is skipped, a violating load reads element 0 of its array, and the violation is recorded
 * on the device.  The ordinary build carries none of these checks.
 */
#ifndef DAB_DEBUG_H
#define DAB_DEBUG_H

#include <stdint.h>

#include "dab.h"

#ifdef __cplusplus
extern "C" {
#endif

typedef struct dab_bounds_report {
  uint64_t violations; /* checked indices found out of range since the last reset */
  int64_t index;       /* the first one recorded ... */
  int64_t extent;      /* ... and the extent it was compared with (valid: 0 <= index < extent) */
  uint32_t file_hash;  /* 32-bit FNV-1a hash of the base name of the source file of that check */
  int32_t line;        /* and its line */
} dab_bounds_report;

/* 1 if this library was built with the checks, 0 otherwise. */
int32_t dab_debug_bounds_enabled(void);

/*
 * Waits for the device (cudaDeviceSynchronize), then writes the sum of the violation records to *h_report
 * (host memory owned by the caller); reset != 0 also clears them.  Returns DAB_ERR_UNSUPPORTED, with
 * *h_report zeroed, from a library built without the checks; DAB_ERR_INVALID_ARG for a null pointer;
 * DAB_ERR_CUDA if the device could not be read.
 */
dab_status dab_debug_bounds_report(dab_bounds_report* h_report, int32_t reset);

#ifdef __cplusplus
}
#endif
#endif
