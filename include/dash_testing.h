/*
 * dash_testing.h -- test hooks of the halted-prefill library (libdash.so).
 *
 * Not part of the product interface (dash.h): entry points that exist so that a test can drive
 * the library into a corner its normal inputs never reach.  Conventions as in dash.h (device
 * pointers, `stream` is a cudaStream_t passed as void*, int status returned).
 */
#ifndef DASH_TESTING_H_
#define DASH_TESTING_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

/* dash_compact (dash.h; the single-pass compaction of Sec. 3.4 / Alg. 1 "gathering tokens") on its
 * look-back path, whatever the size, with a stall planted: the tile ticket starts at 1, so no CTA
 * ever takes tile 0, and tile 1 looks back at a state word that nobody publishes.  Every device-side
 * wait of the library is bounded: after `spin_limit` polls (1 .. 2^22) the waiting tile gives up,
 * sets DASH_ERR_TIMEOUT in the device status word (dash_check_status returns it once and clears it),
 * takes 0 as its base and publishes, so that every later tile finishes and the kernel returns.
 * No row tensors are moved; idx_out [n], cu_out [S+1], n_out_dev as in dash_compact (their contents
 * are unspecified after a timeout; everything written stays inside the buffers).  n >= 64.
 * ws: dash_workspace_bytes(DASH_WS_COMPACT, n, S, ...). */
int dash_testing_compact_stalled(const uint8_t* mask, int64_t n, const int32_t* cu_in, int S,
                                 int32_t* idx_out, int32_t* cu_out, int32_t* n_out_dev,
                                 uint32_t spin_limit, void* ws, size_t ws_bytes, void* stream);

#ifdef __cplusplus
}
#endif
#endif /* DASH_TESTING_H_ */
