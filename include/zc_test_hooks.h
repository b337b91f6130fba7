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
#ifdef __cplusplus
}
#endif
#endif
