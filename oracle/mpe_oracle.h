/*
 * CPU oracle for the mixed-precision cached embedding training step.
 *
 * TEST INFRASTRUCTURE ONLY.  This is a plain, slow, single-threaded C program
 * that restates the method of "Mixed-Precision Embedding using a Cache"
 * (Section 3, Algorithm 1, Algorithm 2, Section 5.1) step by step.  It shares
 * no code with the CUDA library and must never sit on a product path: only
 * tests, the smoke check and the CPU-baseline leg of the benchmark call it.
 *
 * Pins (see tests marked "not gpu"): quantizer closed forms and Algorithm 1
 * idempotence, empirical unbiasedness of stochastic rounding, hand-derived
 * Algorithm 2 tag/priority sequences, the worked de-duplication example of
 * Section 5.1, the full-cache case against a textbook FP32 embedding-bag
 * trainer, a literal single-array emulator of Algorithms 1+2, brute force
 * without a cache, the appendix's memory-compression table; and for the parts
 * the paper does not have -- flush (each resident's entry against the emulator's
 * own quantizer with the flush stream, cache and fetched values unchanged,
 * training identical with and without flushes), ids outside a table (equal to
 * the batch with them deleted), inconsistent offsets (refused, state untouched)
 * and the table mask (equal to a run whose masked tables receive no indices).
 * Parity unpinned (pure conventions, fixed by this build and mirrored on the
 * GPU): the constants of the counter hash, the cache-set hash, INT4 nibble
 * order, argmin tie-breaks, and the radix (32) of the gradient summation tree.
 */
#ifndef MPE_ORACLE_H
#define MPE_ORACLE_H
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

enum { ORC_LRU = 0, ORC_LFU = 1 };
enum { ORC_SGD = 0, ORC_ROWWISE_ADAGRAD = 1 };
enum { ORC_RTN = 0, ORC_SR = 1 };
enum { ORC_DOMAIN_INIT = 1, ORC_DOMAIN_SR = 2, ORC_DOMAIN_FLUSH = 3 };
enum { ORC_OK = 0, ORC_ERR_ARG = -1, ORC_ERR_OFFSETS = -2, ORC_ERR_SEQUENCE = -3 };

typedef struct orc orc;

/* ---- stateless pieces (also used by the pins) --------------------------- */
uint32_t orc_mix32(uint32_t x);
uint32_t orc_rowkey(uint64_t seed, uint32_t domain, uint32_t table, uint32_t row, uint64_t step);
uint32_t orc_draw(uint32_t rowkey, uint32_t column);            /* 32 random bits */
float    orc_uniform(uint32_t rowkey, uint32_t column);         /* (bits>>8)*2^-24 in [0,1) */
uint32_t orc_salt(uint64_t seed, uint32_t table);
int32_t  orc_set_index(uint32_t row, uint32_t salt, int32_t n_sets);
int32_t  orc_num_sets(int64_t num_rows, double cache_fraction, int32_t ways);
/* Row-wise min-max quantizer (Section 3 "Precision", Algorithm 1); codes are
 * written one per byte (unpacked) into q[0..d). */
void orc_quantize(const float* x, int32_t d, int32_t bits, int32_t mode, uint32_t rowkey,
                  uint8_t* q, float* scale, float* bias);
void orc_dequantize(const uint8_t* q, int32_t d, float scale, float bias, float* x);
void orc_pack(const uint8_t* q, int32_t d, int32_t bits, uint8_t* packed);
void orc_unpack(const uint8_t* packed, int32_t d, int32_t bits, uint8_t* q);
/* FP16 table: conversions with a chosen rounding direction (0 nearest-even, 1 toward -inf, 2 toward +inf) and the
 * row-wise down-conversion with nearest or stochastic rounding between the two FP16 neighbours */
float    orc_half_to_float(uint16_t h);
uint16_t orc_float_to_half(float f, int32_t direction);
void orc_to_half_row(const float* x, int32_t d, int32_t mode, uint32_t rowkey, uint16_t* codes16);
void orc_init_row(uint64_t seed, uint32_t table, uint32_t row, int32_t d, float lo, float hi, float* x);
/* Radix-32 summation tree over m rows of d floats (terms[j] points to row j). */
void orc_tree_sum(const float* const* terms, int64_t m, int32_t d, float* out);

/* ---- the stateful step --------------------------------------------------- */
orc* orc_create(const int64_t* num_rows, int32_t num_tables, int32_t dim, int32_t bits,
                double cache_fraction, int32_t ways, int32_t policy, int32_t optimizer,
                float eps, float init_lo, float init_hi, uint64_t seed);
void orc_destroy(orc* o);
/* only tables with table_mask[t] != 0 are processed (NULL = all); lets a test
 * run a sample of the tables of a large configuration */
void orc_set_table_mask(orc* o, const uint8_t* table_mask);
/* rounding used when a row is down-converted during training and flush: ORC_SR (default) or ORC_RTN */
void orc_set_rounding(orc* o, int32_t mode);
int  orc_forward(orc* o, const int32_t* indices, const int32_t* offsets, int32_t batch,
                 int64_t total_indices, float* out);
int  orc_backward(orc* o, const float* grad_out, float lr, int64_t step);
int  orc_flush(orc* o);

/* ---- observation ---------------------------------------------------------- */
int64_t orc_dropped(const orc* o);                /* out-of-range occurrences seen so far */
int32_t orc_sets(const orc* o, int32_t table);
void orc_get_row(orc* o, int32_t table, int64_t row, uint8_t* packed_codes, float* scale, float* bias);
void orc_get_cache(const orc* o, int32_t table, int32_t* tags, float* rows, uint32_t* ts);
uint32_t orc_get_cnt(orc* o, int32_t table, int64_t row);
float    orc_get_adagrad(orc* o, int32_t table, int64_t row);
int64_t  orc_touched(const orc* o, int32_t table, int64_t* rows, int64_t cap);
void orc_stats(const orc* o, int32_t table, uint64_t out8[8]);
void orc_memory_bytes(const orc* o, uint64_t out6[6]);
/* per-unique-row records of the last backward call, in ascending (table,row)
 * order: what the de-duplication produced (Section 5.1) */
int64_t orc_last_unique(const orc* o, int32_t table, int64_t* rows, int32_t* mult, float* grads, int64_t cap);

#ifdef __cplusplus
}
#endif
#endif
