/*
 * shadowsync_profile.h — optional per-kernel timers of the library (measurement aid, no counterpart in the paper).
 *
 * ss_profile(1) makes every kernel launch of the library record a pair of CUDA events around itself on the
 * launching stream; ss_profile(0) switches that off again (the default).  Returns the previous setting.
 * Keep it off while a stream is being captured into a CUDA graph: timing events cannot be read back from
 * a captured launch.
 *
 * ss_profile_collect synchronises the device, then writes one record per timed launch, in launch order:
 * the kernel names, separated by '\n', into names (a host buffer of names_len bytes, NUL-terminated) and
 * the elapsed milliseconds into ms[0..]; at most max_records records.  Returns the number written, or -1
 * if the device could not be synchronised.  The internal list is cleared (call with NULL buffers to discard).
 */
#ifndef SHADOWSYNC_PROFILE_H_
#define SHADOWSYNC_PROFILE_H_
#include <stddef.h>
#ifdef __cplusplus
extern "C" {
#endif
int ss_profile(int on);
int ss_profile_collect(char* names, size_t names_len, float* ms, int max_records);
#ifdef __cplusplus
}
#endif
#endif
