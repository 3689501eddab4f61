/*
 * Entry points that exist only in the checking build of libcstr
 * (libcstr_check.so, compiled with -DCSTR_TESTING -DCSTR_BOUNDS_CHECK).  The
 * release library exports none of them and reads no environment variable.
 * The paper has no counterpart for either: they are test instruments.
 *
 * In the checking build every index that a kernel forms into the DFA table,
 * the token table (next, mask and the builder's intermediate ballot rows), the
 * vocabulary arrays and the logits is compared with the extent of its array
 * before the access.  An index outside its array is recorded in a status
 * record on the device and the access is skipped: no trap, no assert, the
 * kernel runs to its end and the context stays usable.
 */
#ifndef CSTR_DEBUG_H
#define CSTR_DEBUG_H

#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

/*
 * Read the bounds-check record of the current device.
 *   out  HOST uint64 [4]: number of out-of-range indices seen since the last
 *        reset, then for the first of them: the id of the checking site (the
 *        CSTR_SITE_* values of csrc/cstr_internal.cuh), the offending index
 *        and the extent it was compared with
 *   reset  non-zero: clear the record afterwards
 * Synchronises the device.  Returns 0 or a negative CSTR_ERR_* code.
 */
int cstr_debug_bounds_status(uint64_t *out, int32_t reset);

/*
 * Keep only the low `bits` bits (1..63; 0 or 64 = all) of the hash by which
 * the builder's duplicate-column pass groups tokens.  With few bits, tokens of
 * different byte-class strings fall into one group, which exercises the exact
 * comparison that keeps grouping safe.  Affects builds enqueued afterwards.
 */
int cstr_test_set_group_hash_bits(int32_t bits);

#ifdef __cplusplus
}
#endif
#endif /* CSTR_DEBUG_H */
