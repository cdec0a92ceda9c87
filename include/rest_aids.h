/*
 * rest_aids.h - measurement and planning aids of the REST library.  None of these is a step of
 * the method (the paper has no counterpart for any of them); benchmarks and tests use them to
 * explain timings.  The decoding calls are declared in rest.h.
 */
#ifndef REST_AIDS_H_
#define REST_AIDS_H_

#include "rest.h"

#ifdef __cplusplus
extern "C" {
#endif

/*
 * rest_tree_attention_plan - how rest_tree_attention would cut the key range for this shape on
 * the current device (a planning aid; the paper has no counterpart).  out[0] = key ranges per
 * (context, head), out[1] = blocks per cluster (ranges merged on chip), out[2] = clusters per
 * (context, head) (merged through the workspace when > 1), out[3] = clusters of that size the
 * device can run at once.  Host pointers.
 */
rest_status rest_tree_attention_plan(int32_t B, int32_t H, int32_t N, int32_t D, int32_t max_kv,
                                     int32_t* out);

/*
 * rest_probe_dependent_reads - measurement aid (the paper has no counterpart).
 *
 * One device thread follows `steps` dependent loads idx = d_next[idx] from `start` and writes
 * d_out[0] = elapsed nanoseconds (device global timer), d_out[1] = the final index.  With a
 * random cyclic table much larger than L2 this is the latency of one dependent DRAM read; the
 * searches of Algorithm 1 are chains of such reads, so it bounds a single draft from below.
 *   d_next  uint32[n] device table (entries >= n are treated as 0), n <= 2^32 - 1
 *   d_out   uint64[2] device
 */
rest_status rest_probe_dependent_reads(const uint32_t* d_next, uint64_t n, uint32_t start,
                                       uint32_t steps, uint64_t* d_out, void* stream);

/* Number of kernels the library has launched in this process (for launch accounting). */
uint64_t rest_launch_count(void);

#ifdef __cplusplus
}
#endif
#endif /* REST_AIDS_H_ */
