/*
 * CPU oracle for the mixed-precision cached embedding training step.
 * TEST INFRASTRUCTURE ONLY -- see mpe_oracle.h for the role and the pins.
 *
 * Compile with: gcc -O2 -std=c11 -ffp-contract=off -fno-fast-math (no FMA
 * contraction: every fused multiply-add below is an explicit fmaf()).
 *
 * What follows the paper and what is a convention of this build:
 *   - fetch / update operators                      Section 3
 *   - row-wise min-max quantization, (scale, bias)  Section 3 "Precision", Algorithm 1
 *   - nearest-even and stochastic rounding          Section 3 "Rounding"
 *   - n sets x alpha ways, hash h, tags I_C         Section 3 "Cache Structure"
 *   - LFU / LRU priority values, admission rule     Section 3 "Cache Replacement Policy"
 *   - the update loop                               Algorithm 2
 *   - sort + merge of duplicate gradients           Section 5.1
 *   - memory accounting                             Appendix, Eq. 2-3
 *   Conventions (the paper is silent): the counter hash, the set hash, the
 *   order of I_U in Algorithm 2 (hits first, then misses in ascending row id),
 *   timestamps = step number, LFU increment = multiplicity in the batch, the
 *   radix-32 gradient summation tree, row-wise Adagrad's formula, and the
 *   multiplication by 1/scale instead of a division per element.
 */
#include "mpe_oracle.h"

#include <float.h>
#include <math.h>
#include <stdlib.h>
#include <string.h>

/* ------------------------------------------------------------------------ */
/* Counter-based hash (convention).  All arithmetic is modulo 2^32.          */
/* ------------------------------------------------------------------------ */
uint32_t orc_mix32(uint32_t x) {
    x ^= x >> 16;
    x *= 0x7feb352dU;
    x ^= x >> 15;
    x *= 0x846ca68bU;
    x ^= x >> 16;
    return x;
}

static uint32_t absorb(uint32_t h, uint32_t w) { return orc_mix32((h ^ w) + 0x9E3779B9U); }

uint32_t orc_rowkey(uint64_t seed, uint32_t domain, uint32_t table, uint32_t row, uint64_t step) {
    uint32_t h = 0x243F6A88U;
    h = absorb(h, (uint32_t)(seed & 0xFFFFFFFFU));
    h = absorb(h, (uint32_t)(seed >> 32));
    h = absorb(h, domain);
    h = absorb(h, table);
    h = absorb(h, row);
    h = absorb(h, (uint32_t)(step & 0xFFFFFFFFU));
    h = absorb(h, (uint32_t)(step >> 32));
    return h;
}

uint32_t orc_draw(uint32_t rowkey, uint32_t column) {
    return orc_mix32(rowkey ^ (column * 0x9E3779B9U + 0x7F4A7C15U));
}

float orc_uniform(uint32_t rowkey, uint32_t column) {
    return (float)(orc_draw(rowkey, column) >> 8) * 0x1p-24f; /* exact: 24-bit integer times 2^-24 */
}

uint32_t orc_salt(uint64_t seed, uint32_t table) {
    uint32_t h = 0x13198A2EU;
    h = absorb(h, (uint32_t)(seed & 0xFFFFFFFFU));
    h = absorb(h, (uint32_t)(seed >> 32));
    h = absorb(h, table);
    return h;
}

/* h : {0..N-1} -> {0..n-1}  (Section 3 "Cache Structure"; the function itself is a convention) */
int32_t orc_set_index(uint32_t row, uint32_t salt, int32_t n_sets) {
    uint64_t m = (uint64_t)orc_mix32(row ^ salt) * (uint64_t)(uint32_t)n_sets;
    return (int32_t)(m >> 32);
}

/* number of sets: the cache never exceeds fraction*N rows; at least one set when fraction > 0 */
int32_t orc_num_sets(int64_t num_rows, double cache_fraction, int32_t ways) {
    if (!(cache_fraction > 0.0)) return 0;
    int64_t cache_rows = (int64_t)floor(cache_fraction * (double)num_rows + 1e-6);
    int64_t n = cache_rows / ways;
    if (n < 1) n = 1;
    return (int32_t)n;
}

/* ------------------------------------------------------------------------ */
/* Quantizer (Section 3 "Precision" / "Rounding", Algorithm 1)               */
/* ------------------------------------------------------------------------ */
void orc_quantize(const float* x, int32_t d, int32_t bits, int32_t mode, uint32_t rowkey,
                  uint8_t* q, float* scale, float* bias) {
    float mn = x[0], mx = x[0];
    for (int c = 1; c < d; ++c) {
        mn = fminf(mn, x[c]);
        mx = fmaxf(mx, x[c]);
    }
    mn = mn + 0.0f;                              /* -0 becomes +0: bias bits independent of scan order */
    const float qmax = (float)((1 << bits) - 1); /* 2^N - 1 */
    float s = (mx - mn) / qmax;                  /* s = (max - min)/(2^N - 1) */
    float inv = 0.0f;
    if (s >= FLT_MIN) inv = 1.0f / s;
    if (inv == 0.0f) s = 0.0f;                   /* constant row: every code 0, bias carries the value */
    for (int c = 0; c < d; ++c) {
        float y = (x[c] - mn) * inv;             /* (x - b)/s */
        y = fminf(fmaxf(y, 0.0f), qmax);
        int code;
        if (mode == ORC_RTN) {
            code = (int)rintf(y);                /* round to nearest, ties to even */
        } else {
            float f = floorf(y);
            float p = y - f;                     /* exact */
            float u = orc_uniform(rowkey, (uint32_t)c);
            code = (int)f + (u < p ? 1 : 0);     /* x+ with probability p, x- otherwise: E = y */
        }
        q[c] = (uint8_t)code;
    }
    *scale = s;
    *bias = mn;
}

void orc_dequantize(const uint8_t* q, int32_t d, float scale, float bias, float* x) {
    for (int c = 0; c < d; ++c) x[c] = fmaf((float)q[c], scale, bias); /* q*s + b */
}

/* 8/bits codes per byte, lowest column in the lowest bits (INT4: column 2k in the low nibble of byte k) */
void orc_pack(const uint8_t* q, int32_t d, int32_t bits, uint8_t* packed) {
    const int per = 8 / bits, mask = (1 << bits) - 1;
    for (int k = 0; k < d / per; ++k) {
        unsigned v = 0;
        for (int j = 0; j < per; ++j) v |= (unsigned)(q[per * k + j] & mask) << (bits * j);
        packed[k] = (uint8_t)v;
    }
}

void orc_unpack(const uint8_t* packed, int32_t d, int32_t bits, uint8_t* q) {
    const int per = 8 / bits, mask = (1 << bits) - 1;
    for (int k = 0; k < d / per; ++k)
        for (int j = 0; j < per; ++j) q[per * k + j] = (uint8_t)((packed[k] >> (bits * j)) & mask);
}

/* ------------------------------------------------------------------------ */
/* FP16 table (Section 3 "Precision"/"Rounding": the two neighbours of x in    */
/* FP16 differ by one unit in the last place)                                 */
/* ------------------------------------------------------------------------ */
float orc_half_to_float(uint16_t h) {
    const int sign = h >> 15, e = (h >> 10) & 31, m = h & 1023;
    float v;
    if (e == 0) v = ldexpf((float)m, -24);                   /* zero and subnormals: m * 2^-24 */
    else if (e == 31) v = m ? NAN : INFINITY;
    else v = ldexpf((float)(m | 1024), e - 25);              /* 1.m * 2^(e-15) */
    return sign ? -v : v;
}

/* FP32 -> FP16 with a chosen rounding direction: 0 nearest-even, 1 toward -inf, 2 toward +inf */
uint16_t orc_float_to_half(float f, int32_t direction) {
    uint32_t bits;
    memcpy(&bits, &f, 4);
    const uint32_t sign = bits >> 31, exp = (bits >> 23) & 255, man = bits & 0x7FFFFF;
    if (exp == 255) return (uint16_t)((sign << 15) | 0x7C00 | (man ? 0x200 : 0));
    /* |f| = m24 * 2^(e-23); FP32 subnormals are far below the smallest FP16 step and only leave a sticky bit */
    const uint32_t m24 = exp ? (man | 0x800000) : man;
    const int e = exp ? (int)exp - 127 : -126;
    uint32_t h, rem, half_point;
    if (e > 15) {                                             /* beyond the FP16 range (the caller clamps before) */
        h = 0x7BFF; rem = 1; half_point = 0;
    } else if (e >= -14) {                                    /* normal FP16: keep 11 of the 24 significand bits */
        h = ((uint32_t)(e + 15) << 10) | ((m24 >> 13) & 1023);
        rem = m24 & 0x1FFF; half_point = 0x1000;
    } else {                                                  /* subnormal FP16: multiples of 2^-24 */
        const int shift = 13 + (-14 - e);
        if (shift >= 32) { h = 0; rem = m24 ? 1 : 0; half_point = 2; }
        else { h = m24 >> shift; rem = m24 & ((1u << shift) - 1); half_point = 1u << (shift - 1); }
    }
    int up;                                                   /* whether the magnitude moves to the next code */
    if (direction == 0) up = rem > half_point || (rem == half_point && rem != 0 && (h & 1));
    else if (direction == 1) up = sign && rem != 0;
    else up = !sign && rem != 0;
    if (up) h += 1;                                           /* a carry runs into the exponent field, as it should */
    return (uint16_t)((sign << 15) | h);
}

/* down-convert one row to FP16; codes16[c] receives the half-precision bits */
void orc_to_half_row(const float* x, int32_t d, int32_t mode, uint32_t rowkey, uint16_t* codes16) {
    for (int c = 0; c < d; ++c) {
        const float v = fminf(fmaxf(x[c], -65504.0f), 65504.0f);      /* stay inside the finite FP16 range */
        if (mode == ORC_RTN) { codes16[c] = orc_float_to_half(v, 0); continue; }
        const uint16_t lo = orc_float_to_half(v, 1), hi = orc_float_to_half(v, 2);    /* x- <= x <= x+ */
        if (lo == hi) { codes16[c] = lo; continue; }
        const float flo = orc_half_to_float(lo), fhi = orc_half_to_float(hi);
        const float p = (v - flo) / (fhi - flo);                  /* exact: both differences fit FP32, the step is a power of two */
        codes16[c] = orc_uniform(rowkey, (uint32_t)c) < p ? hi : lo;  /* x+ with probability p: expectation x */
    }
}

void orc_init_row(uint64_t seed, uint32_t table, uint32_t row, int32_t d, float lo, float hi, float* x) {
    uint32_t key = orc_rowkey(seed, ORC_DOMAIN_INIT, table, row, 0);
    float width = hi - lo;
    for (int c = 0; c < d; ++c) x[c] = fmaf(orc_uniform(key, (uint32_t)c), width, lo);
}

/* ------------------------------------------------------------------------ */
/* Duplicate-gradient merge (Section 5.1): radix-32 summation tree            */
/* ------------------------------------------------------------------------ */
void orc_tree_sum(const float* const* terms, int64_t m, int32_t d, float* out) {
    if (m <= 32) {
        for (int c = 0; c < d; ++c) out[c] = terms[0][c];
        for (int64_t j = 1; j < m; ++j)
            for (int c = 0; c < d; ++c) out[c] = out[c] + terms[j][c];
        return;
    }
    int64_t nchunk = (m + 31) / 32;
    float* sums = (float*)malloc((size_t)nchunk * (size_t)d * sizeof(float));
    const float** ptr = (const float**)malloc((size_t)nchunk * sizeof(float*));
    for (int64_t k = 0; k < nchunk; ++k) {
        int64_t len = m - 32 * k < 32 ? m - 32 * k : 32;
        orc_tree_sum(terms + 32 * k, len, d, sums + k * d);
        ptr[k] = sums + k * d;
    }
    orc_tree_sum(ptr, nchunk, d, out);
    free(ptr);
    free(sums);
}

/* ------------------------------------------------------------------------ */
/* State                                                                     */
/* ------------------------------------------------------------------------ */
typedef struct {
    int64_t N;
    int32_t n_sets;
    uint32_t salt;
    /* low-precision table T, materialised lazily: an untouched row is the
     * pure function init(seed, table, row) quantized with nearest-even */
    int64_t* hkey; int64_t* hval; int64_t hcap, nrec, rcap;
    int64_t* rec_row;
    uint8_t* codes;   /* nrec x code_bytes (packed) */
    float* scale; float* bias;
    uint32_t* cnt;    /* LFU access counters, one per embedding row */
    float* G;         /* row-wise Adagrad accumulator */
    /* cache C: n sets x alpha ways */
    int32_t* tag;     /* I_C; -1 = empty */
    float* crow;      /* FP32 rows */
    uint32_t* ts;     /* LRU timestamps (0 = never) */
    uint64_t stats[8];
    /* last backward's unique rows (observation only) */
    int64_t nu; int64_t* u_row; int32_t* u_mult; float* u_grad;
} table_t;

struct orc {
    int32_t T, d, bits, ways, policy, optimizer, code_bytes;
    double cache_fraction;
    float eps, lo, hi;
    uint64_t seed;
    table_t* tb;
    uint8_t* mask;
    /* inputs of the last forward, kept for backward */
    int32_t* indices; int32_t* offsets; int32_t batch; int64_t total; int have_forward;
    int64_t dropped;
    int64_t last_step;
    int32_t rounding;   /* how update() down-converts: ORC_SR (default) or ORC_RTN (Section 3 "Rounding") */
};

static uint64_t hash64(int64_t k) {
    uint64_t x = (uint64_t)k;
    x ^= x >> 33; x *= 0xff51afd7ed558ccdULL; x ^= x >> 33; x *= 0xc4ceb9fe1a85ec53ULL; x ^= x >> 33;
    return x;
}

static int64_t rec_find(const table_t* tb, int64_t row) {
    uint64_t i = hash64(row) & (uint64_t)(tb->hcap - 1);
    while (tb->hkey[i] != -1) {
        if (tb->hkey[i] == row) return tb->hval[i];
        i = (i + 1) & (uint64_t)(tb->hcap - 1);
    }
    return -1;
}

static void map_put(table_t* tb, int64_t row, int64_t val) {
    uint64_t i = hash64(row) & (uint64_t)(tb->hcap - 1);
    while (tb->hkey[i] != -1) i = (i + 1) & (uint64_t)(tb->hcap - 1);
    tb->hkey[i] = row;
    tb->hval[i] = val;
}

static void initial_row(const orc* o, int32_t t, int64_t row, uint8_t* packed, float* s, float* b) {
    float x[1024];
    uint8_t q[1024];
    orc_init_row(o->seed, (uint32_t)t, (uint32_t)row, o->d, o->lo, o->hi, x);
    if (o->bits == 16) { orc_to_half_row(x, o->d, ORC_RTN, 0, (uint16_t*)packed); *s = 1.0f; *b = 0.0f; return; }
    orc_quantize(x, o->d, o->bits, ORC_RTN, 0, q, s, b);
    orc_pack(q, o->d, o->bits, packed);
}

/* record id of a row, materialising it on first touch */
static int64_t rec_get(orc* o, int32_t t, int64_t row) {
    table_t* tb = &o->tb[t];
    int64_t id = rec_find(tb, row);
    if (id >= 0) return id;
    if (tb->nrec == tb->rcap) {
        tb->rcap *= 2;
        tb->rec_row = (int64_t*)realloc(tb->rec_row, (size_t)tb->rcap * sizeof(int64_t));
        tb->codes = (uint8_t*)realloc(tb->codes, (size_t)tb->rcap * (size_t)o->code_bytes);
        tb->scale = (float*)realloc(tb->scale, (size_t)tb->rcap * sizeof(float));
        tb->bias = (float*)realloc(tb->bias, (size_t)tb->rcap * sizeof(float));
        tb->cnt = (uint32_t*)realloc(tb->cnt, (size_t)tb->rcap * sizeof(uint32_t));
        tb->G = (float*)realloc(tb->G, (size_t)tb->rcap * sizeof(float));
    }
    if ((tb->nrec + 1) * 2 > tb->hcap) {
        int64_t oldcap = tb->hcap;
        int64_t* ok = tb->hkey; int64_t* ov = tb->hval;
        tb->hcap *= 2;
        tb->hkey = (int64_t*)malloc((size_t)tb->hcap * sizeof(int64_t));
        tb->hval = (int64_t*)malloc((size_t)tb->hcap * sizeof(int64_t));
        for (int64_t i = 0; i < tb->hcap; ++i) tb->hkey[i] = -1;
        for (int64_t i = 0; i < oldcap; ++i) if (ok[i] != -1) map_put(tb, ok[i], ov[i]);
        free(ok); free(ov);
    }
    id = tb->nrec++;
    tb->rec_row[id] = row;
    initial_row(o, t, row, tb->codes + id * o->code_bytes, &tb->scale[id], &tb->bias[id]);
    tb->cnt[id] = 0;
    tb->G[id] = 0.0f;
    map_put(tb, row, id);
    return id;
}

orc* orc_create(const int64_t* num_rows, int32_t num_tables, int32_t dim, int32_t bits,
                double cache_fraction, int32_t ways, int32_t policy, int32_t optimizer,
                float eps, float init_lo, float init_hi, uint64_t seed) {
    if (num_tables < 1 || dim < 4 || dim > 1024 || (dim & (dim - 1)) != 0) return NULL;
    if (bits != 8 && bits != 4 && bits != 2 && bits != 16) return NULL;
    if (ways == 0) ways = 32;
    if (ways < 1 || ways > 32 || (ways & (ways - 1)) != 0) return NULL;
    if (!(cache_fraction >= 0.0 && cache_fraction <= 1.0)) return NULL;
    orc* o = (orc*)calloc(1, sizeof(orc));
    o->T = num_tables; o->d = dim; o->bits = bits; o->ways = ways; o->policy = policy;
    o->optimizer = optimizer; o->code_bytes = dim * bits / 8; o->cache_fraction = cache_fraction;
    o->eps = eps; o->lo = init_lo; o->hi = init_hi; o->seed = seed; o->rounding = ORC_SR;
    o->tb = (table_t*)calloc((size_t)num_tables, sizeof(table_t));
    for (int t = 0; t < num_tables; ++t) {
        table_t* tb = &o->tb[t];
        tb->N = num_rows[t];
        tb->n_sets = orc_num_sets(tb->N, cache_fraction, ways);
        tb->salt = orc_salt(seed, (uint32_t)t);
        tb->hcap = 1024; tb->rcap = 256; tb->nrec = 0;
        tb->hkey = (int64_t*)malloc((size_t)tb->hcap * sizeof(int64_t));
        tb->hval = (int64_t*)malloc((size_t)tb->hcap * sizeof(int64_t));
        for (int64_t i = 0; i < tb->hcap; ++i) tb->hkey[i] = -1;
        tb->rec_row = (int64_t*)malloc((size_t)tb->rcap * sizeof(int64_t));
        tb->codes = (uint8_t*)malloc((size_t)tb->rcap * (size_t)o->code_bytes);
        tb->scale = (float*)malloc((size_t)tb->rcap * sizeof(float));
        tb->bias = (float*)malloc((size_t)tb->rcap * sizeof(float));
        tb->cnt = (uint32_t*)malloc((size_t)tb->rcap * sizeof(uint32_t));
        tb->G = (float*)malloc((size_t)tb->rcap * sizeof(float));
        int64_t slots = (int64_t)tb->n_sets * ways;
        tb->tag = (int32_t*)malloc((size_t)(slots > 0 ? slots : 1) * sizeof(int32_t));
        tb->crow = (float*)calloc((size_t)(slots > 0 ? slots : 1) * (size_t)dim, sizeof(float));
        tb->ts = (uint32_t*)calloc((size_t)(slots > 0 ? slots : 1), sizeof(uint32_t));
        for (int64_t i = 0; i < slots; ++i) tb->tag[i] = -1;
    }
    return o;
}

void orc_destroy(orc* o) {
    if (!o) return;
    for (int t = 0; t < o->T; ++t) {
        table_t* tb = &o->tb[t];
        free(tb->hkey); free(tb->hval); free(tb->rec_row); free(tb->codes); free(tb->scale);
        free(tb->bias); free(tb->cnt); free(tb->G); free(tb->tag); free(tb->crow); free(tb->ts);
        free(tb->u_row); free(tb->u_mult); free(tb->u_grad);
    }
    free(o->tb); free(o->mask); free(o->indices); free(o->offsets);
    free(o);
}

void orc_set_rounding(orc* o, int32_t mode) { o->rounding = mode == ORC_RTN ? ORC_RTN : ORC_SR; }

void orc_set_table_mask(orc* o, const uint8_t* table_mask) {
    free(o->mask);
    o->mask = NULL;
    if (table_mask) {
        o->mask = (uint8_t*)malloc((size_t)o->T);
        memcpy(o->mask, table_mask, (size_t)o->T);
    }
}

/* way of `row` in its set, or -1 */
static int find_way(const orc* o, const table_t* tb, int32_t set, int64_t row) {
    for (int w = 0; w < o->ways; ++w)
        if (tb->tag[(int64_t)set * o->ways + w] == (int32_t)row) return w;
    return -1;
}

/* fetch(T, C, i)  (Section 3): the FP32 cache row if resident, else the up-converted low-precision row */
static void fetch(orc* o, int32_t t, int64_t row, float* x) {
    table_t* tb = &o->tb[t];
    if (tb->n_sets > 0) {
        int32_t set = orc_set_index((uint32_t)row, tb->salt, tb->n_sets);
        int w = find_way(o, tb, set, row);
        if (w >= 0) {
            memcpy(x, tb->crow + ((int64_t)set * o->ways + w) * o->d, (size_t)o->d * sizeof(float));
            return;
        }
    }
    int64_t id = rec_get(o, t, row);
    uint8_t q[1024];
    if (o->bits == 16) {   /* FP16 table: the up-conversion is exact */
        const uint16_t* hrow = (const uint16_t*)(tb->codes + id * o->code_bytes);
        for (int c = 0; c < o->d; ++c) x[c] = orc_half_to_float(hrow[c]);
        return;
    }
    orc_unpack(tb->codes + id * o->code_bytes, o->d, o->bits, q);
    orc_dequantize(q, o->d, tb->scale[id], tb->bias[id], x);
}

/* down-convert x into T[row] with the rounding method of choice (stochastic unless set otherwise) */
static void store_quantized(orc* o, int32_t t, int64_t row, const float* x, uint32_t domain, int64_t step) {
    table_t* tb = &o->tb[t];
    int64_t id = rec_get(o, t, row);
    uint8_t q[1024];
    uint32_t key = orc_rowkey(o->seed, domain, (uint32_t)t, (uint32_t)row, (uint64_t)step);
    if (o->bits == 16) { orc_to_half_row(x, o->d, o->rounding, key, (uint16_t*)(tb->codes + id * o->code_bytes)); return; }
    orc_quantize(x, o->d, o->bits, o->rounding, key, q, &tb->scale[id], &tb->bias[id]);
    orc_pack(q, o->d, o->bits, tb->codes + id * o->code_bytes);
}

static int offsets_ok(const int32_t* offsets, int64_t nbags, int64_t total) {
    if (offsets[0] != 0 || offsets[nbags] != total) return 0;
    for (int64_t i = 0; i < nbags; ++i) if (offsets[i + 1] < offsets[i]) return 0;
    return 1;
}

/* ------------------------------------------------------------------------ */
/* Forward: fetch every index of every bag and sum-pool (state is read only)  */
/* ------------------------------------------------------------------------ */
int orc_forward(orc* o, const int32_t* indices, const int32_t* offsets, int32_t batch,
                int64_t total_indices, float* out) {
    if (!o || batch < 0 || total_indices < 0) return ORC_ERR_ARG;
    const int64_t nbags = (int64_t)o->T * batch;
    if (!offsets_ok(offsets, nbags, total_indices)) return ORC_ERR_OFFSETS;
    const int d = o->d;
    float x[1024];
    for (int t = 0; t < o->T; ++t) {
        if (o->mask && !o->mask[t]) continue;
        for (int b = 0; b < batch; ++b) {
            float* acc = out + ((int64_t)b * o->T + t) * d;
            for (int c = 0; c < d; ++c) acc[c] = 0.0f;
            const int64_t bag = (int64_t)t * batch + b;
            for (int64_t p = offsets[bag]; p < offsets[bag + 1]; ++p) {
                int64_t row = indices[p];
                if (row < 0 || row >= o->tb[t].N) { o->dropped++; continue; }
                fetch(o, t, row, x);
                for (int c = 0; c < d; ++c) acc[c] = acc[c] + x[c];
            }
        }
    }
    free(o->indices); free(o->offsets);
    o->indices = (int32_t*)malloc((size_t)(total_indices > 0 ? total_indices : 1) * sizeof(int32_t));
    o->offsets = (int32_t*)malloc((size_t)(nbags + 1) * sizeof(int32_t));
    memcpy(o->indices, indices, (size_t)total_indices * sizeof(int32_t));
    memcpy(o->offsets, offsets, (size_t)(nbags + 1) * sizeof(int32_t));
    o->batch = batch; o->total = total_indices; o->have_forward = 1;
    return ORC_OK;
}

/* ------------------------------------------------------------------------ */
/* Backward: de-duplicate, merge gradients, update, run Algorithm 2           */
/* ------------------------------------------------------------------------ */
typedef struct { int64_t row; int64_t p; } occ_t;

static int occ_cmp(const void* a, const void* b) {
    const occ_t* x = (const occ_t*)a; const occ_t* y = (const occ_t*)b;
    if (x->row != y->row) return x->row < y->row ? -1 : 1;
    if (x->p != y->p) return x->p < y->p ? -1 : 1;
    return 0;
}

/* priority value PV of the resident in (set, way); empty ways rank below everything */
static int64_t resident_pv(orc* o, int32_t t, int32_t set, int w) {
    table_t* tb = &o->tb[t];
    int64_t slot = (int64_t)set * o->ways + w;
    if (tb->tag[slot] < 0) return -1;
    if (o->policy == ORC_LFU) return (int64_t)tb->cnt[rec_get(o, t, tb->tag[slot])];
    return (int64_t)tb->ts[slot];
}

static void optimizer_step(const orc* o, table_t* tb, int64_t id, const float* x, const float* g, float lr, float* xn) {
    const int d = o->d;
    if (o->optimizer == ORC_SGD) {
        for (int c = 0; c < d; ++c) xn[c] = fmaf(-lr, g[c], x[c]);   /* x <- x - eta * dL/dx */
        return;
    }
    /* row-wise Adagrad: G += mean(g^2); x <- x - lr/(sqrt(G)+eps) * g.
     * Sum of squares: four consecutive elements per partial (fmaf chain),
     * partials combined by a halving-stride binary tree. */
    float P[256];
    const int nl = d / 4;
    for (int l = 0; l < nl; ++l) {
        float a = g[4 * l] * g[4 * l];
        a = fmaf(g[4 * l + 1], g[4 * l + 1], a);
        a = fmaf(g[4 * l + 2], g[4 * l + 2], a);
        a = fmaf(g[4 * l + 3], g[4 * l + 3], a);
        P[l] = a;
    }
    for (int stride = nl / 2; stride >= 1; stride /= 2)
        for (int l = 0; l < stride; ++l) P[l] = P[l] + P[l + stride];
    tb->G[id] = tb->G[id] + P[0] * (1.0f / (float)d);
    float mult = lr / (sqrtf(tb->G[id]) + o->eps);
    for (int c = 0; c < d; ++c) xn[c] = fmaf(-mult, g[c], x[c]);
}

int orc_backward(orc* o, const float* grad_out, float lr, int64_t step) {
    if (!o) return ORC_ERR_ARG;
    if (!o->have_forward) return ORC_ERR_SEQUENCE;
    if (step < 1 || step <= o->last_step || step > 0xFFFFFFFFLL) return ORC_ERR_ARG;
    const int d = o->d, B = o->batch, A = o->ways;
    for (int t = 0; t < o->T; ++t) {
        if (o->mask && !o->mask[t]) continue;
        table_t* tb = &o->tb[t];
        /* --- sort the occurrences of this table by (row, position): Section 5.1 --- */
        const int64_t p0 = o->offsets[(int64_t)t * B], p1 = o->offsets[(int64_t)(t + 1) * B];
        occ_t* occ = (occ_t*)malloc((size_t)(p1 - p0 + 1) * sizeof(occ_t));
        int32_t* bag_of = (int32_t*)malloc((size_t)(p1 - p0 + 1) * sizeof(int32_t));
        int64_t n = 0;
        for (int b = 0; b < B; ++b)
            for (int64_t p = o->offsets[(int64_t)t * B + b]; p < o->offsets[(int64_t)t * B + b + 1]; ++p) {
                bag_of[p - p0] = b;
                int64_t row = o->indices[p];
                if (row < 0 || row >= tb->N) continue;   /* dropped occurrence (counted in forward) */
                occ[n].row = row; occ[n].p = p; ++n;
            }
        qsort(occ, (size_t)n, sizeof(occ_t), occ_cmp);
        int64_t nu = 0;
        for (int64_t i = 0; i < n; ++i) if (i == 0 || occ[i].row != occ[i - 1].row) ++nu;
        /* --- unique rows, multiplicities, merged gradients --- */
        int64_t* urow = (int64_t*)malloc((size_t)(nu + 1) * sizeof(int64_t));
        int32_t* umult = (int32_t*)malloc((size_t)(nu + 1) * sizeof(int32_t));
        float* ug = (float*)malloc((size_t)(nu + 1) * (size_t)d * sizeof(float));
        float* xnew = (float*)malloc((size_t)(nu + 1) * (size_t)d * sizeof(float));
        int8_t* was_hit = (int8_t*)malloc((size_t)(nu + 1));
        int64_t k = 0;
        for (int64_t i = 0; i < n;) {
            int64_t j = i;
            while (j < n && occ[j].row == occ[i].row) ++j;
            const int64_t m = j - i;
            const float** terms = (const float**)malloc((size_t)m * sizeof(float*));
            for (int64_t a = 0; a < m; ++a)   /* ascending position: the sort is stable by construction */
                terms[a] = grad_out + ((int64_t)bag_of[occ[i + a].p - p0] * o->T + t) * d;
            orc_tree_sum(terms, m, d, ug + k * d);
            free(terms);
            urow[k] = occ[i].row; umult[k] = (int32_t)m;
            ++k; i = j;
        }
        tb->stats[0] += (uint64_t)n;
        tb->stats[2] += (uint64_t)nu;
        /* --- Algorithm 2, with I_U ordered: all hits first, then misses in ascending row id --- */
        /* priority values first: every row of I_U is now one access more popular / more recent (Section 3 "Cache Replacement Policy") */
        for (k = 0; k < nu; ++k) {
            const int64_t row = urow[k];
            int w = -1; int32_t set = 0;
            if (tb->n_sets > 0) { set = orc_set_index((uint32_t)row, tb->salt, tb->n_sets); w = find_way(o, tb, set, row); }
            was_hit[k] = (int8_t)(w >= 0);
            if (o->policy == ORC_LFU) {
                int64_t id = rec_get(o, t, row);
                uint64_t c = (uint64_t)tb->cnt[id] + (uint64_t)umult[k];
                tb->cnt[id] = c > 0xFFFFFFFFULL ? 0xFFFFFFFFU : (uint32_t)c;   /* access count */
            } else if (w >= 0) {
                tb->ts[(int64_t)set * A + w] = (uint32_t)step;                 /* last-access timestamp */
            }
            if (w >= 0) { tb->stats[1] += (uint64_t)umult[k]; tb->stats[3] += 1; }
        }
        /* the gradient update itself, in full precision, applied to the value the forward fetched (Section 3 "update") */
        float x[1024];
        for (k = 0; k < nu; ++k) {
            fetch(o, t, urow[k], x);
            optimizer_step(o, tb, rec_get(o, t, urow[k]), x, ug + k * d, lr, xnew + k * d);
        }
        /* hits: the row is cache resident, overwrite it in the cache */
        for (k = 0; k < nu; ++k) {
            if (!was_hit[k]) continue;
            int32_t set = orc_set_index((uint32_t)urow[k], tb->salt, tb->n_sets);
            int w = find_way(o, tb, set, urow[k]);
            memcpy(tb->crow + ((int64_t)set * A + w) * d, xnew + k * d, (size_t)d * sizeof(float));
        }
        /* misses: bypass or replace */
        for (k = 0; k < nu; ++k) {
            if (was_hit[k]) continue;
            const int64_t row = urow[k];
            if (tb->n_sets == 0) {   /* no cache at all: pure low-precision training (Algorithm 1) */
                store_quantized(o, t, row, xnew + k * d, ORC_DOMAIN_SR, step);
                continue;
            }
            const int32_t set = orc_set_index((uint32_t)row, tb->salt, tb->n_sets);
            const int64_t pv_i = o->policy == ORC_LFU ? (int64_t)tb->cnt[rec_get(o, t, row)] : step;
            int j = 0; int64_t pv_j = resident_pv(o, t, set, 0);
            for (int w = 1; w < A; ++w) {   /* the resident of lowest priority value in the set; ties -> lowest way */
                int64_t pv = resident_pv(o, t, set, w);
                if (pv < pv_j) { pv_j = pv; j = w; }
            }
            int bypass = pv_i <= pv_j;
            if (A == 1 && o->policy == ORC_LRU) bypass = 0;   /* direct-mapped LRU always replaces */
            const int64_t slot = (int64_t)set * A + j;
            if (bypass) {
                store_quantized(o, t, row, xnew + k * d, ORC_DOMAIN_SR, step);
                tb->stats[6] += 1;
            } else {
                if (tb->tag[slot] >= 0) {   /* evicted row is down-converted and placed back in T */
                    store_quantized(o, t, tb->tag[slot], tb->crow + slot * d, ORC_DOMAIN_SR, step);
                    tb->stats[5] += 1;
                }
                tb->tag[slot] = (int32_t)row;                 /* the newcomer takes over the tag */
                memcpy(tb->crow + slot * d, xnew + k * d, (size_t)d * sizeof(float));   /* verbatim */
                if (o->policy == ORC_LRU) tb->ts[slot] = (uint32_t)step;
                tb->stats[4] += 1;
            }
        }
        tb->stats[7] += 1;
        free(tb->u_row); free(tb->u_mult); free(tb->u_grad);
        tb->nu = nu; tb->u_row = urow; tb->u_mult = umult; tb->u_grad = ug;
        free(xnew); free(was_hit); free(occ); free(bag_of);
    }
    o->last_step = step;
    o->have_forward = 0;
    return ORC_OK;
}

/* every resident row is down-converted into T and stays resident (snapshot) */
int orc_flush(orc* o) {
    if (!o) return ORC_ERR_ARG;
    for (int t = 0; t < o->T; ++t) {
        if (o->mask && !o->mask[t]) continue;
        table_t* tb = &o->tb[t];
        const int64_t slots = (int64_t)tb->n_sets * o->ways;
        for (int64_t s = 0; s < slots; ++s)
            if (tb->tag[s] >= 0) store_quantized(o, t, tb->tag[s], tb->crow + s * o->d, ORC_DOMAIN_FLUSH, o->last_step);
    }
    return ORC_OK;
}

/* ------------------------------------------------------------------------ */
/* Observation                                                               */
/* ------------------------------------------------------------------------ */
int64_t orc_dropped(const orc* o) { return o->dropped; }
int32_t orc_sets(const orc* o, int32_t table) { return o->tb[table].n_sets; }

void orc_get_row(orc* o, int32_t table, int64_t row, uint8_t* packed_codes, float* scale, float* bias) {
    table_t* tb = &o->tb[table];
    int64_t id = rec_find(tb, row);
    if (id < 0) { initial_row(o, table, row, packed_codes, scale, bias); return; }
    memcpy(packed_codes, tb->codes + id * o->code_bytes, (size_t)o->code_bytes);
    *scale = tb->scale[id]; *bias = tb->bias[id];
}

void orc_get_cache(const orc* o, int32_t table, int32_t* tags, float* rows, uint32_t* ts) {
    const table_t* tb = &o->tb[table];
    const int64_t slots = (int64_t)tb->n_sets * o->ways;
    if (tags) memcpy(tags, tb->tag, (size_t)slots * sizeof(int32_t));
    if (rows) memcpy(rows, tb->crow, (size_t)slots * (size_t)o->d * sizeof(float));
    if (ts) memcpy(ts, tb->ts, (size_t)slots * sizeof(uint32_t));
}

uint32_t orc_get_cnt(orc* o, int32_t table, int64_t row) {
    int64_t id = rec_find(&o->tb[table], row);
    return id < 0 ? 0U : o->tb[table].cnt[id];
}

float orc_get_adagrad(orc* o, int32_t table, int64_t row) {
    int64_t id = rec_find(&o->tb[table], row);
    return id < 0 ? 0.0f : o->tb[table].G[id];
}

int64_t orc_touched(const orc* o, int32_t table, int64_t* rows, int64_t cap) {
    const table_t* tb = &o->tb[table];
    for (int64_t i = 0; i < tb->nrec && i < cap; ++i) rows[i] = tb->rec_row[i];
    return tb->nrec;
}

void orc_stats(const orc* o, int32_t table, uint64_t out8[8]) {
    memcpy(out8, o->tb[table].stats, 8 * sizeof(uint64_t));
}

/* Appendix Eq. 2-3: bytes of each component (M_Q is inside the low-precision table size) */
void orc_memory_bytes(const orc* o, uint64_t out6[6]) {
    uint64_t lowprec = 0, cache = 0, tags = 0, pv = 0, opt = 0, fp32 = 0;
    for (int t = 0; t < o->T; ++t) {
        const uint64_t N = (uint64_t)o->tb[t].N, slots = (uint64_t)o->tb[t].n_sets * (uint64_t)o->ways;
        lowprec += N * ((uint64_t)o->bits * (uint64_t)o->d + (o->bits == 16 ? 0 : 64)) / 8;   /* E x (bitwidth x D + 64) bits; FP16 has no scale/bias */
        cache += slots * 4 * (uint64_t)o->d;                            /* 4 alpha n d bytes */
        tags += slots * 4;                                              /* INT32 per cached row */
        if (slots > 0) pv += o->policy == ORC_LFU ? N * 4 : slots * 4;  /* INT32 counter per embedding row (LFU) */
        if (o->optimizer == ORC_ROWWISE_ADAGRAD) opt += N * 4;
        fp32 += N * 4 * (uint64_t)o->d;
    }
    out6[0] = lowprec; out6[1] = cache; out6[2] = tags; out6[3] = pv; out6[4] = opt; out6[5] = fp32;
}

int64_t orc_last_unique(const orc* o, int32_t table, int64_t* rows, int32_t* mult, float* grads, int64_t cap) {
    const table_t* tb = &o->tb[table];
    for (int64_t i = 0; i < tb->nu && i < cap; ++i) {
        if (rows) rows[i] = tb->u_row[i];
        if (mult) mult[i] = tb->u_mult[i];
        if (grads) memcpy(grads + i * o->d, tb->u_grad + i * o->d, (size_t)o->d * sizeof(float));
    }
    return tb->nu;
}
