/*
 * sva_debug.h -- test and tuning aids exported by libsva.so next to the public calls of sva.h.
 *
 * Unlike everything in sva.h these three calls keep PROCESS-GLOBAL state (two host variables and one device
 * variable per loaded library): a setting stays in force for every later attention launch of the process
 * until it is set back.  They are meant for single-threaded test and bench programs.  The paper has no
 * counterpart.
 */
#ifndef SVA_DEBUG_H_
#define SVA_DEBUG_H_

#ifdef __cplusplus
extern "C" {
#endif

/*
 * Cycle counter of the attention kernel.  buf: DEVICE buffer of at least 320 int64 (the caller zeroes it), or
 * NULL to switch the counter off again.  While set, every attention launch does an atomicMax of its CTAs'
 * elapsed SM cycles (clock64 from kernel entry to tear-down) into buf[319]: the cycle count of the longest
 * CTA, i.e. of the launch, independent of the SM clock (cycles / time = the clock the launch really ran at).
 */
void sva_debug_set_prof_buffer(void* buf);

/*
 * Kernel behaviour switches for the next attention launches (0 = normal operation).
 *   bit 0: skip the exponentials (tuning aid: timing only, results are wrong);
 *   bit 4: test aid: the K producer withholds a row's tiles after the first, so that a bounded pipeline wait
 *          runs out and the kernel takes its give-up path (SVA_DEV_TIMEOUT) -- nothing faults or hangs.
 *   bit 5: measurement aid: bf16 attention reads V where it lies (MN-major operand) instead of the transposed copy;
 *   bit 7: test aid: the remainder call masks the kept blocks of a block-mean tile by looking them up in the CSR
 *          (the form that serves more than 1024 key blocks) even where the kept-block bit masks would serve.
 */
void sva_debug_set_mode(int bits);

/*
 * Test aid: the number of SM cycles a device-side wait may last before its CTA gives up (default 3e9;
 * cycles <= 0 restores the default).  Synchronous (a small host-to-device copy on the current device).
 * Returns 0 on success.
 */
int sva_debug_set_wait_limit(long long cycles);

#ifdef __cplusplus
}
#endif
#endif /* SVA_DEBUG_H_ */
