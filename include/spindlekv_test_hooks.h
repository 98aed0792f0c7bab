/*
 * spindlekv_test_hooks.h -- knobs and self-tests for the test suite of the SpindleKV reduction library.
 *
 * None of this belongs to the paper's calls (spindlekv.h).  The library bounds every device-side wait
 * and every data-dependent loop, and it prefers a compact candidate list to the adjacency bit matrix
 * as long as the list fits.  The limits involved are generous by default, so ordinary inputs never reach
 * them; the functions below let a test tighten them, so that the paths behind the limits (a wait or a loop that
 * gives up and reports SPINDLEKV_TIMEOUT, a unit that falls back to the bit matrix) can be exercised
 * without ever hanging or faulting a GPU.  The settings are process-wide and are read when a call is
 * issued; they are not meant for production use.
 */
#ifndef SPINDLEKV_TEST_HOOKS_H_
#define SPINDLEKV_TEST_HOOKS_H_

#include "spindlekv.h"

#ifdef __cplusplus
extern "C" {
#endif

enum {
  SPINDLEKV_TUNE_RECORDS_PER_TILE = 0,  /* candidate records a row block of the similarity kernel may write per 128 x 256
                                           tile (default 512, the most the workspace is sized for); 0: no candidate
                                           records, every unit is computed as a bit matrix */
  SPINDLEKV_TUNE_GREEDY_ROUND_CAP = 1,  /* rounds after which the greedy cover gives up (default: the sequence length,
                                           which an exact run can never exceed) */
  SPINDLEKV_TUNE_MBAR_WAIT_CYCLES = 2,  /* SM clock cycles after which a wait on a shared-memory barrier of the
                                           tensor-core kernels gives up */
  SPINDLEKV_TUNE_SIM_BLOCK_PAIRS = 3    /* pairs of blocks the candidate-record similarity kernel runs on (default 0:
                                           as many as the device holds at once); fewer make every pair walk more
                                           (unit, row span) items one after the other */
};

/* Sets one limit; value < 0 restores its default.  INVALID_ARG for an unknown key. */
spindlekv_status spindlekv_set_tuning(int32_t key, int64_t value);
/* Current value of a limit, or -1 for an unknown key. */
int64_t spindlekv_get_tuning(int32_t key);

/*
 * Self-test of the bounded wait of the tensor-core kernels: launches one small kernel on `stream` in which a
 * block waits on a shared-memory barrier on which nobody ever arrives, with a limit short enough to run out at
 * once (`limit`: SM clock cycles).  The kernel must return by itself and leave SPINDLEKV_TIMEOUT in the status
 * word at the start of `ws` (device, at least 256 bytes, 256-byte aligned; cleared by the call), which
 * spindlekv_poll_status then reports.
 */
spindlekv_status spindlekv_selftest_mbarrier_timeout(void* ws, int64_t limit, void* stream);

#ifdef __cplusplus
}
#endif
#endif /* SPINDLEKV_TEST_HOOKS_H_ */
