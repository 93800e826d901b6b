/*
 * shadowsync_harness.h — device-side generator of synthetic embedding tables.
 *
 * Not part of the method: it only fills a table with the counter-based uniform values that define
 * the synthetic workloads, so that a table of tens of GB never has to exist on the host.
 *
 *   dst[i] = ((u >> 8) * 2^-24 - 0.5) * scale + mid,   u = high 32 bits of mix64(key + (counter0 + i + 1) * GAMMA)
 *
 * with mix64 the SplitMix64 output function and GAMMA = 0x9E3779B97F4A7C15; every float operation
 * is rounded to nearest separately, so the host generator reproduces the values bit for bit.
 * dst: device float[count].  Returns SS_OK or a negative ss_status (see shadowsync.h).
 */
#ifndef SHADOWSYNC_HARNESS_H_
#define SHADOWSYNC_HARNESS_H_
#include "shadowsync.h"
#ifdef __cplusplus
extern "C" {
#endif
ss_status ssh_fill_uniform(float* dst, int64_t count, uint64_t key, uint64_t counter0, float scale, float mid,
                           ss_stream stream);
#ifdef __cplusplus
}
#endif
#endif
