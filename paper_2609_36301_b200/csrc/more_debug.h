/*
 * Diagnostic entry points of libmore_route.so.  Not part of the public interface (include/more_route.h): they exist
 * for the test-suite and for the instrumented builds, and may change without notice.
 */
#ifndef MORE_DEBUG_H_
#define MORE_DEBUG_H_

#ifdef __cplusplus
extern "C" {
#endif

/*
 * more_route_debug_counters -- synchronise `stream`, copy the current device's 16 epilogue event counters to out16
 * (host) and clear them.  The kernels only maintain the counters when the library was built with -DMORE_STATS;
 * otherwise they read zero.
 */
int more_route_debug_counters(unsigned long long* out16, void* stream);

/*
 * more_debug_expire_wait -- launch a one-warp kernel that waits, with the library's bounded mbarrier wait, on a barrier
 * nobody ever arrives at, with a budget of `budget_cycles` SM clocks (a millisecond or so is plenty).  The wait runs out
 * by construction, the kernel records MORE_ERR_TIMEOUT in the device status word exactly as the router kernels would,
 * and returns normally: nothing hangs, traps or faults.  The next more_route_status() must report MORE_ERR_TIMEOUT once.
 * No TMA, no tensor memory.  Asynchronous on `stream`.
 */
int more_debug_expire_wait(long long budget_cycles, void* stream);

/*
 * more_debug_scratch_guard -- the library's cached scratch allocation carries a 256-byte guard region behind the bytes
 * the last plan asked for, filled with a pattern when the plan is made.  This call synchronises `stream` and returns 1
 * if the guard still holds the pattern, 0 if something wrote into it, or a negative MORE_ERR_* code.
 */
int more_debug_scratch_guard(void* stream);

#ifdef __cplusplus
}
#endif
#endif /* MORE_DEBUG_H_ */
