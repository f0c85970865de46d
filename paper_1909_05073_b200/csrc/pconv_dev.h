/*
 * Development entry points of the PCONV library.  They exist only in a library compiled with
 * -DPCONV_DEV (build.py: build(dev=True) -> libpconv_dev.so) and are not part of the public ABI
 * in include/pconv.h; none has a counterpart in the paper.  The development build is otherwise the
 * same code: it adds phase timestamps to the tiled kernel, lets the environment force a launch
 * plan (PCONV_FORCE_ZS / PCONV_FORCE_KS), and can make one bounded wait of a launch run out so
 * that the give-up path -- status word, skipped work, common exit, Tensor Memory handed back --
 * can be exercised without faulting or hanging anything.
 */
#ifndef PCONV_DEV_H_
#define PCONV_DEV_H_

#include "../../include/pconv.h"

#ifdef __cplusplus
extern "C" {
#endif

/* Synchronises the device and copies the first n_words (<= PCONV_TRACE_WORDS) 64-bit trace words
 * of the handle to the HOST: timestamps of the tiled kernel's phases (nanoseconds of the global
 * timer for words 0-10, SM cycles for 11-12; each word's meaning is listed where the kernel
 * writes it). */
#define PCONV_TRACE_WORDS 14
pconv_status pconv_trace_read(const pconv_handle* h, unsigned long long* words_host, int n_words);

/* From now on, in every tiled-kernel launch on the current device, one producer thread leaves out
 * its arrival for chunk `chunk` (counted inside a CTA's chunk range) on the stage's "full"
 * barrier, and every bounded wait gives up after `spin_limit` tries (each try suspends the warp
 * for at most 200 ns) instead of the normal limit.  The consumers of that chunk then run out of
 * patience, record wait id 2 in the status word, skip their remaining work and leave through the
 * common exit; the launch produces no valid output.  chunk < 0 switches the behaviour off and
 * restores the normal limit.  Synchronises the device. */
pconv_status pconv_dev_withhold(int chunk, unsigned spin_limit);

/* Clears the handle's sticky status word (pconv_device_status reports PCONV_OK again until the
 * next abandoned wait).  Synchronises the device. */
pconv_status pconv_dev_clear_status(const pconv_handle* h);

#ifdef __cplusplus
}
#endif
#endif /* PCONV_DEV_H_ */
