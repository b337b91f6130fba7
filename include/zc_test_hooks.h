/*
 * zc_test_hooks.h — host-side entry points that exist only so the word-level field split and
 * merge used by the kernels (the same inline functions, compiled for the host) can be checked
 * on a machine without a GPU.  They are not part of the product path and are never called by it.
 * The operations are the field split / merge of Sec. 3.1, 3.2 and 3.4 of the paper and the byte
 * grouping of its Fig. 7 caption, on one 16-byte group of elements (8 symbols per stream).
 */
#ifndef ZC_TEST_HOOKS_H
#define ZC_TEST_HOOKS_H
#include "zc.h"
#ifdef __cplusplus
extern "C" {
#endif
/* h_in16: 16 element bytes (host).  h_e8 / h_sm8: receive 8 exponent symbols / 8 sign+mantissa
 * symbols.  Returns ZC_E_UNSUPPORTED for an unknown format, ZC_E_INVALID_ARG for null pointers. */
zc_status zc_test_split16(zc_format fmt, const uint8_t* h_in16, uint8_t* h_e8, uint8_t* h_sm8);
/* Inverse: 8 + 8 symbols (host) -> 16 element bytes (host). */
zc_status zc_test_merge16(zc_format fmt, const uint8_t* h_e8, const uint8_t* h_sm8, uint8_t* h_out16);

/* ---- bounded waits (no counterpart in the paper: failure handling of this library) ----------
 * Every wait inside a kernel (for another block's look-back word, for a batch inside a block,
 * for the bulk copy of a chunk's piece) gives up after a number of polls and the call reports
 * ZC_E_DEVICE_TIMEOUT.  These switches let a test reach that branch without hanging or faulting
 * anything: the kernels return by themselves.  They change process-wide settings; a test puts
 * them back (polls = 0 restores the default limit, 0 turns a stall off).
 *   zc_test_set_wait_limit  polls after which a device-side wait gives up
 *   zc_test_stall_encoder   zc_compress hands out its batches from this number on, so batch 0 is
 *                           never packed and every look-back waits for a word nobody posts
 *   zc_test_stall_decoder   the decoder does not start the copies of the pieces it waits for */
/* Launch shapes (host arithmetic only, no GPU): worker warps per block the encoder would use for a plan
 * with n_coded Huffman-coded streams (0..2) and pack slots of class wide_slots (0: 8 bits per symbol, 1: 12 bits,
 * 2: one slot of 4 bits per symbol, which the library picks for chunks from 16 KiB whose codes are short), and warps
 * per block of the decoder with one or both streams coded.  0 = the kernels cannot take this plan.  A test checks
 * that every chunk size zc_plan accepts gives at least one. */
uint32_t zc_test_encoder_workers(const zc_plan_t* plan, uint32_t n_coded, uint32_t wide_slots);
uint32_t zc_test_decoder_warps(const zc_plan_t* plan, uint32_t both_coded);
void zc_test_set_wait_limit(uint32_t polls);
void zc_test_stall_encoder(uint32_t first_ticket);
void zc_test_stall_decoder(uint32_t on);
/* Development build of the library (compiled with -DZC_DEBUG_CHECKS=1): every shared-memory and global-memory
 * access the kernels make through their load/store helpers is checked against the block's shared window and the
 * buffers of the launch; a violation is counted and the access skipped (no trap, no fault).  This call waits for the
 * device, stores the number of refused shared accesses in out[0] and of refused global accesses in out[1], clears
 * the counters and returns 1.  The ordinary build has no checks: it returns 0 and leaves out alone. */
int zc_test_debug_counts(uint32_t out[2]);
#ifdef __cplusplus
}
#endif
#endif
