/* monde_diagnostics.h -- diagnostic and test switches of libmonde.so.
 *
 * None of these is part of the layer (the paper has no counterpart for them); they exist so
 * that tests and measurements can reach code paths that normal use selects by itself or never
 * takes.  They are PROCESS-WIDE state, read when a call of include/monde.h enqueues its kernels:
 * set them while no other thread is calling the library.  With every switch at its default the
 * library behaves exactly as include/monde.h describes.
 */
#ifndef MONDE_DIAGNOSTICS_H_
#define MONDE_DIAGNOSTICS_H_

#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

/* Expert FFN on CTA pairs (clusters of two CTAs, one 256-row tcgen05.mma per pair) instead of
 * single CTAs.  mode: 1 = pairs, 0 = single CTAs, negative = the library's default (single CTAs).
 * Both modes compute the same sums in the same order. */
void monde_diag_set_ffn_cta_pairs(int mode);

/* Per-unit device timeline of the expert FFN kernel.  `device_buf`: device memory for
 * (number of SMs) * slots * 8 uint64 values, owned by the caller and kept alive while the switch
 * is on; NULL or slots <= 0 switches the timeline off (the default).  Per CTA and unit slot:
 * unit id, producer first / last issue, first operands ready, accumulator committed, epilogue
 * start / end (global timer, ns). */
void monde_diag_set_trace(void* device_buf, int slots);

/* Bound of every device-side wait (mbarrier phases, dependency counters), in nanoseconds;
 * 0 restores the default of 2 s.  A wait on another unit's results gives up after this long and
 * the waits inside a CTA, which can only be waiting for that one, after twice as long; the kernel
 * then records MONDE_ERR_TIMEOUT and returns (see monde_poll_device_status). */
void monde_diag_set_wait_limit_ns(unsigned long long ns);

/* on = 1: first-layer units of the expert FFN finish without publishing their hidden rows, so
 * that every second-layer unit's wait for them runs out.  Used with a short wait limit to
 * exercise the give-up path: all accesses stay in bounds, the kernel returns by itself with
 * MONDE_ERR_TIMEOUT recorded and y_perm undefined.  0 (default): normal operation. */
void monde_diag_set_hold_hidden_ready(int on);

/* Number of one-time set-up steps (function attributes for large dynamic shared memory) that
 * have run on CUDA device `device` in this process: they run once per device, with that device
 * current, at the first call that needs them.  -1 for a device index outside 0..63. */
int monde_diag_device_setups(int device);

/* Range checks.  A library built with -DMONDE_DIAGNOSTICS (`python -m paper_2405_18832_b200.build
 * --diagnostics` makes libmonde_diag.so) checks every index its kernels take from memory before using
 * it as an address: expert ids and positions in the permutation, positions in the combine, the rows
 * and features of every work unit of the expert FFN.  A value out of range is counted, the first one
 * is kept with a site code (1 permute expert id, 2 permute position, 3 combine position, 4 FFN unit
 * rows, 5 FFN unit features), and the access is skipped; an FFN unit out of range also records
 * MONDE_ERR_BOUNDS in the workspace.  It stands in for a memory checker where none may be run.
 * This call synchronises the device, returns the number of violations since the last call and
 * clears the record; `first_site` / `first_value` (nullable, host pointers) receive the first one.
 * Returns -1 from a library that was not built with the checks, -2 if the record cannot be read. */
int monde_diag_bounds_violations(int32_t* first_site, long long* first_value);

#ifdef __cplusplus
}
#endif
#endif /* MONDE_DIAGNOSTICS_H_ */
