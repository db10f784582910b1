/*
 * TAH-Quant boundary codec -- CPU ORACLE (test infrastructure, not the product).
 *
 * A plain, slow, scalar restatement of the method of "TAH-Quant: Effective
 * Activation Quantization in Pipeline Parallelism over Slow Network"
 * (Sec. 3.1-3.4, Eq. 1-4, Algorithm 1 lines 4-5).  It exists so that the CUDA
 * library can be checked against something written independently from the
 * paper.  Only the test-suite, the smoke check and the benchmark's CPU
 * baseline may call it; the CUDA library never does and shares no code,
 * header, table or helper with it.
 *
 * All pointers are HOST pointers.  All arithmetic that decides a stored bit
 * is IEEE-754 binary32, round-to-nearest-even, evaluated in exactly the order
 * written in tahq_oracle.c (compile with -ffp-contract=off).
 */
#ifndef TAHQ_ORACLE_H
#define TAHQ_ORACLE_H

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

enum { TAHQO_F32 = 0, TAHQO_BF16 = 1 };

typedef struct {
  uint32_t dtype;            /* TAHQO_F32 / TAHQO_BF16, dense row-major [tokens x hidden]        */
  uint64_t tokens;           /* T = B*S                                                            */
  uint32_t hidden;           /* C, a multiple of tile                                              */
  uint32_t group_tokens;     /* S: tokens per ranking group ("sample", Sec. 3.2); 0 means T        */
  uint32_t tile;             /* G (= A, the default of Sec. 3.2): power of two, 8..128             */
  uint32_t budget_millibits; /* payload bits per element x 1000, 2000..8000                        */
  float tau;                 /* outlier threshold of Eq. 3 (paper: 2.0)                            */
  float eps_l1;              /* epsilon of Eq. 1                                                   */
  float eps_log;             /* varsigma of Eq. 2                                                  */
  float eps_ratio;           /* varrho of Eq. 3                                                    */
  uint32_t rounding;         /* 0 = round-half-even, 1 = stochastic (Philox4x32-10)                */
  uint64_t seed;             /* key of the stochastic-rounding stream                              */
  uint32_t alloc_tile;       /* A of Sec. 3.2: allocation-tile width, a multiple of tile that divides
                                hidden; 0 means A = G (the paper's default); A = hidden is token-level   */
} tahqo_params;

/* Section offsets of the packed buffer (bytes from its start). */
typedef struct {
  uint64_t n_tiles, n_groups, tiles_per_group, k_hi;   /* k_hi counts quantisation tiles per group */
  uint32_t lo_bits, hi_bits;
  uint64_t off_bitmap, off_scale_zero, off_pivot, off_payload;
  uint64_t payload_bytes, total_bytes;
} tahqo_layout;

/* 0 on success, non-zero when the parameters are not a valid configuration. */
int tahqo_layout_of(const tahqo_params *p, tahqo_layout *out);
size_t tahqo_packed_bound(const tahqo_params *p);

/* Whole-tensor encode / decode.  Return 0 on success. */
int tahqo_encode(const tahqo_params *p, const void *in, uint8_t *packed, size_t packed_cap);
int tahqo_decode(const tahqo_params *p, const uint8_t *packed, size_t packed_bytes, void *out);

/* Per-step entry points, exported so that the tests can pin each step alone. */
float tahqo_treesum(const float *x, uint32_t n);                       /* fixed pairwise tree, any n */
void tahqo_lg2_array(const float *x, float *y, size_t n);             /* the oracle's log2        */
float tahqo_score(const float *tile, uint32_t G, float eps_l1, float eps_log); /* Eq. 1-2         */
void tahqo_allocate(const float *score, uint64_t n, uint64_t k_hi, uint8_t *is_hi); /* Sec. 3.2   */
void tahqo_pivot(const float *tile, uint32_t G, float tau, float eps_ratio,
                 uint32_t *d, int *flag);                              /* Eq. 3                    */
void tahqo_swap_hadamard(float *tile, uint32_t G, uint32_t d);         /* Eq. 4 (in place)         */
uint16_t tahqo_f32_to_f16(float x);
float tahqo_f16_to_f32(uint16_t h);
uint16_t tahqo_f32_to_bf16(float x);
void tahqo_range(const float *v, uint32_t G, uint32_t bits, uint16_t *s_h, uint16_t *z_h);
void tahqo_quantise(const float *v, uint32_t G, uint32_t bits, uint16_t s_h, uint16_t z_h,
                    uint32_t rounding, uint64_t seed, uint64_t first_elem, uint32_t *q);
void tahqo_philox4x32_10(const uint32_t key[2], const uint32_t ctr[4], uint32_t out[4]);

#ifdef __cplusplus
}
#endif
#endif
