/*
 * Fixed-point ("naive") gradient compressor -- CPU ORACLE (test infrastructure, not the product).
 *
 * The backward half of Algorithm 1 (lines 6-7): the gradient with respect to the boundary
 * activations travels through a simple fixed-point quantiser of 6-10 bits (Sec. 3.5), optionally
 * pre-scaled by a constant c, g_hat = Q(c g) / c (appendix, "Gradient scaling").  The paper gives
 * no formula for Q_Naive; the reading implemented here is stated step by step in qnaive_oracle.c.
 * All pointers are HOST pointers.
 */
#ifndef QNAIVE_ORACLE_H
#define QNAIVE_ORACLE_H

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef struct {
  uint32_t dtype;       /* 0 = binary32, 1 = bfloat16; dense row-major [tokens x hidden]       */
  uint64_t tokens;
  uint32_t hidden;      /* a multiple of 8                                                    */
  uint32_t bits;        /* b in [2, 16]                                                       */
  uint32_t per_tensor;  /* 0: one scale per token (row); 1: one scale for the whole tensor    */
  float prescale;       /* c > 0, finite                                                      */
} qnaiveo_params;

typedef struct {
  uint64_t n_scales, off_scales, off_payload, row_bytes, total_bytes;
} qnaiveo_layout;

int qnaiveo_layout_of(const qnaiveo_params *p, qnaiveo_layout *out);
size_t qnaiveo_packed_bound(const qnaiveo_params *p);
int qnaiveo_encode(const qnaiveo_params *p, const void *in, uint8_t *packed, size_t cap);
int qnaiveo_decode(const qnaiveo_params *p, const uint8_t *packed, size_t bytes, void *out);

#ifdef __cplusplus
}
#endif
#endif
