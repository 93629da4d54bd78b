/*
 * bt_oracle.c -- TEST INFRASTRUCTURE ONLY (see bt_oracle.h).
 *
 * Every loop walks one element (one bit) at a time in the order the paper's
 * Algorithms 1 and 2 state; there is no blocking, vectorisation or threading.
 * Where the paper leaves a point open the reading taken is written beside it.
 */
#include "bt_oracle.h"
#include <string.h>

#define CHUNK_ELEMS 4096u

int oracle_elem_size(int kind)
{
    switch (kind) {
    case ORACLE_F32:  return 4;
    case ORACLE_F16:  return 2;
    case ORACLE_BF16: return 2;
    case ORACLE_F64:  return 8;
    default:          return 0;
    }
}

/* "T[i] == 0" of Algorithm 1 is read as "every byte of the element is zero":
 * -0.0, NaN, infinities and subnormals are non-zero and are stored verbatim,
 * which is what makes the round trip bitwise lossless. */
static int all_bytes_zero(const unsigned char *p, int elem_size)
{
    for (int b = 0; b < elem_size; ++b)
        if (p[b] != 0) return 0;
    return 1;
}

/* Algorithm 1: scan the flattened tensor; push a 0 bit for a zero, else push
 * the element to the values vector and push a 1 bit. The chunk prefix entry is
 * the count of values pushed so far, taken whenever i reaches a multiple of 4096. */
uint64_t oracle_compress(const void *dense, uint64_t n, int elem_size,
                         uint32_t *bitmap, void *values, uint64_t *prefix)
{
    const unsigned char *src = (const unsigned char *)dense;
    unsigned char *val = (unsigned char *)values;
    uint64_t words = (n + 31) / 32;
    uint64_t j = 0;

    for (uint64_t w = 0; w < words; ++w) bitmap[w] = 0;     /* padding bits stay 0 */

    for (uint64_t i = 0; i < n; ++i) {                      /* half-open: 0 <= i < n */
        if (i % CHUNK_ELEMS == 0) prefix[i / CHUNK_ELEMS] = j;
        const unsigned char *e = src + i * (uint64_t)elem_size;
        if (all_bytes_zero(e, elem_size)) {
            /* push 0 bit: already 0 */
        } else {
            memcpy(val + j * (uint64_t)elem_size, e, (size_t)elem_size);   /* push T[i] */
            j += 1;
            bitmap[i >> 5] |= (uint32_t)1 << (i & 31);                     /* push 1 bit */
        }
    }
    return j;
}

/* Algorithm 2: j = 0; for every bit, a set bit takes values[j] and advances j,
 * a clear bit yields 0.0 (all-zero bytes in every precision). */
void oracle_decompress(const uint32_t *bitmap, const void *values,
                       uint64_t n, int elem_size, void *dense_out)
{
    const unsigned char *val = (const unsigned char *)values;
    unsigned char *dst = (unsigned char *)dense_out;
    uint64_t j = 0;
    for (uint64_t i = 0; i < n; ++i) {
        unsigned char *e = dst + i * (uint64_t)elem_size;
        if ((bitmap[i >> 5] >> (i & 31)) & 1u) {
            memcpy(e, val + j * (uint64_t)elem_size, (size_t)elem_size);
            j += 1;
        } else {
            memset(e, 0, (size_t)elem_size);
        }
    }
}

void oracle_decompress_chunked(const uint32_t *bitmap, const void *values,
                               const uint64_t *prefix, uint64_t n, int elem_size,
                               void *dense_out)
{
    const unsigned char *val = (const unsigned char *)values;
    unsigned char *dst = (unsigned char *)dense_out;
    uint64_t chunks = (n + CHUNK_ELEMS - 1) / CHUNK_ELEMS;
    for (uint64_t c = 0; c < chunks; ++c) {
        uint64_t j = prefix[c];                               /* restart the counter */
        uint64_t lo = c * CHUNK_ELEMS;
        uint64_t hi = lo + CHUNK_ELEMS < n ? lo + CHUNK_ELEMS : n;
        for (uint64_t i = lo; i < hi; ++i) {
            unsigned char *e = dst + i * (uint64_t)elem_size;
            if ((bitmap[i >> 5] >> (i & 31)) & 1u) {
                memcpy(e, val + j * (uint64_t)elem_size, (size_t)elem_size);
                j += 1;
            } else {
                memset(e, 0, (size_t)elem_size);
            }
        }
    }
}

/* binary16 -> binary32, exact (every half is representable as a float). */
float oracle_half_to_float(uint16_t h)
{
    uint32_t sign = (uint32_t)(h >> 15) & 1u;
    uint32_t expo = (uint32_t)(h >> 10) & 0x1Fu;
    uint32_t mant = (uint32_t)h & 0x3FFu;
    uint32_t out;
    if (expo == 0x1Fu) {                       /* inf or NaN: keep the payload */
        out = (sign << 31) | 0x7F800000u | (mant << 13);
    } else if (expo != 0) {                    /* normal: rebias 15 -> 127 */
        out = (sign << 31) | ((expo + 112u) << 23) | (mant << 13);
    } else if (mant == 0) {                    /* signed zero */
        out = sign << 31;
    } else {                                   /* subnormal: value = mant * 2^-24 */
        float f = (float)mant * (1.0f / 16777216.0f);
        if (sign) f = -f;
        return f;
    }
    float f;
    memcpy(&f, &out, 4);
    return f;
}

/* Is this element "<= 0" under IEEE comparison?  (false for NaN) */
static int le_zero(const unsigned char *e, int kind)
{
    switch (kind) {
    case ORACLE_F32: { float f; memcpy(&f, e, 4); return f <= 0.0f; }
    case ORACLE_F64: { double d; memcpy(&d, e, 8); return d <= 0.0; }
    case ORACLE_F16: { uint16_t h; memcpy(&h, e, 2); return oracle_half_to_float(h) <= 0.0f; }
    case ORACLE_BF16: {                        /* bfloat16 is the top half of a binary32 */
        uint16_t h; memcpy(&h, e, 2);
        uint32_t u = (uint32_t)h << 16; float f; memcpy(&f, &u, 4);
        return f <= 0.0f;
    }
    default: return 0;
    }
}

/* ReLU is where the sparsity comes from (section 3.1); the activation is
 * stashed in the forward pass (section 3.2).  y = (x <= 0) ? +0 : x, so -0,
 * negatives and -inf become +0 (all-zero bytes), positives are raw copies and
 * a NaN stays a NaN with its payload.  Then Algorithm 1 on y. */
uint64_t oracle_relu_fwd_compress(const void *pre_act, uint64_t n, int kind,
                                  void *y, uint32_t *bitmap, void *values,
                                  uint64_t *prefix)
{
    int elem_size = oracle_elem_size(kind);
    const unsigned char *src = (const unsigned char *)pre_act;
    unsigned char *yo = (unsigned char *)y;
    unsigned char *val = (unsigned char *)values;
    uint64_t words = (n + 31) / 32;
    uint64_t j = 0;
    unsigned char act[8];

    for (uint64_t w = 0; w < words; ++w) bitmap[w] = 0;

    for (uint64_t i = 0; i < n; ++i) {
        if (i % CHUNK_ELEMS == 0) prefix[i / CHUNK_ELEMS] = j;
        const unsigned char *e = src + i * (uint64_t)elem_size;
        if (le_zero(e, kind)) memset(act, 0, (size_t)elem_size);
        else                  memcpy(act, e, (size_t)elem_size);
        if (yo) memcpy(yo + i * (uint64_t)elem_size, act, (size_t)elem_size);
        if (!all_bytes_zero(act, elem_size)) {
            memcpy(val + j * (uint64_t)elem_size, act, (size_t)elem_size);
            j += 1;
            bitmap[i >> 5] |= (uint32_t)1 << (i & 31);
        }
    }
    return j;
}

/* Is this element "<= tau" under IEEE comparison?  (false for NaN)  The element is
 * widened exactly (binary16 / bfloat16 -> binary32, binary64 stays, tau widens
 * to binary64), so the decision is taken on exact values of both sides. */
static int le_tau(const unsigned char *e, int kind, float tau)
{
    switch (kind) {
    case ORACLE_F32: { float f; memcpy(&f, e, 4); return f <= tau; }
    case ORACLE_F64: { double d; memcpy(&d, e, 8); return d <= (double)tau; }
    case ORACLE_F16: { uint16_t h; memcpy(&h, e, 2); return oracle_half_to_float(h) <= tau; }
    case ORACLE_BF16: {
        uint16_t h; memcpy(&h, e, 2);
        uint32_t u = (uint32_t)h << 16; float f; memcpy(&f, &u, 4);
        return f <= tau;
    }
    default: return 0;
    }
}

/* Activation pruning joined to the stash (section 4, "Combining BitTrain with
 * Activation Pruning"): only activations that exceed a close-to-zero threshold
 * tau are stored, the others are taken to be zero.  y = (x <= tau) ? +0 : x --
 * "exceeds" read as a strict comparison, so that tau = 0 is the ReLU above, and
 * a NaN, which neither exceeds nor falls below anything, is kept.  Then
 * Algorithm 1 on y. */
uint64_t oracle_prune_fwd_compress(const void *x, uint64_t n, int kind, float tau,
                                   void *y, uint32_t *bitmap, void *values,
                                   uint64_t *prefix)
{
    int elem_size = oracle_elem_size(kind);
    const unsigned char *src = (const unsigned char *)x;
    unsigned char *yo = (unsigned char *)y;
    unsigned char *val = (unsigned char *)values;
    uint64_t words = (n + 31) / 32;
    uint64_t j = 0;
    unsigned char act[8];

    for (uint64_t w = 0; w < words; ++w) bitmap[w] = 0;

    for (uint64_t i = 0; i < n; ++i) {
        if (i % CHUNK_ELEMS == 0) prefix[i / CHUNK_ELEMS] = j;
        const unsigned char *e = src + i * (uint64_t)elem_size;
        if (le_tau(e, kind, tau)) memset(act, 0, (size_t)elem_size);
        else                      memcpy(act, e, (size_t)elem_size);
        if (yo) memcpy(yo + i * (uint64_t)elem_size, act, (size_t)elem_size);
        if (!all_bytes_zero(act, elem_size)) {
            memcpy(val + j * (uint64_t)elem_size, act, (size_t)elem_size);
            j += 1;
            bitmap[i >> 5] |= (uint32_t)1 << (i & 31);
        }
    }
    return j;
}

/* Double-mask batch normalisation (section 3.1: the zero pattern of the
 * normalisation layer's INPUT is applied as a mask to its OUTPUT, which carries
 * the sparsity through the layer).  The mask is the bitmap the input's stash
 * already holds, so the output's stash reuses it and only needs the vector of
 * values: walk the elements as Algorithm 1 does, but push x[i] where bit i of
 * the mask is 1 -- whatever x[i] is -- instead of testing x[i].  y, when asked
 * for, is the masked dense tensor.  Returns the number of values pushed (the
 * number of set bits among the first n). */
uint64_t oracle_mask_compress(const void *x, uint64_t n, int elem_size,
                              const uint32_t *mask_bitmap, void *y, void *values)
{
    const unsigned char *src = (const unsigned char *)x;
    unsigned char *yo = (unsigned char *)y;
    unsigned char *val = (unsigned char *)values;
    uint64_t j = 0;
    for (uint64_t i = 0; i < n; ++i) {
        const unsigned char *e = src + i * (uint64_t)elem_size;
        if ((mask_bitmap[i >> 5] >> (i & 31)) & 1u) {
            memcpy(val + j * (uint64_t)elem_size, e, (size_t)elem_size);
            j += 1;
            if (yo) memcpy(yo + i * (uint64_t)elem_size, e, (size_t)elem_size);
        } else if (yo) {
            memset(yo + i * (uint64_t)elem_size, 0, (size_t)elem_size);
        }
    }
    return j;
}

/* Compare an element with 6 after exact widening: sets *ge6 (x >= 6) and *lt6
 * (x < 6); both are 0 for a NaN. */
static void cmp_six(const unsigned char *e, int kind, int *ge6, int *lt6)
{
    double d = 0.0;
    switch (kind) {
    case ORACLE_F32: { float f; memcpy(&f, e, 4); d = (double)f; break; }
    case ORACLE_F64: { memcpy(&d, e, 8); break; }
    case ORACLE_F16: { uint16_t h; memcpy(&h, e, 2); d = (double)oracle_half_to_float(h); break; }
    case ORACLE_BF16: {
        uint16_t h; memcpy(&h, e, 2);
        uint32_t u = (uint32_t)h << 16; float f; memcpy(&f, &u, 4); d = (double)f; break;
    }
    default: break;
    }
    *ge6 = d >= 6.0;
    *lt6 = d < 6.0;
}

/* the value 6 in the element type (exact in all four) */
static void six_pattern(int kind, unsigned char *out)
{
    switch (kind) {
    case ORACLE_F32: { float f = 6.0f; memcpy(out, &f, 4); break; }
    case ORACLE_F64: { double d = 6.0; memcpy(out, &d, 8); break; }
    case ORACLE_F16: { uint16_t h = 0x4600; memcpy(out, &h, 2); break; }     /* 1.5 * 2^2 */
    case ORACLE_BF16: { uint16_t h = 0x40C0; memcpy(out, &h, 2); break; }    /* top half of 0x40C00000 */
    default: break;
    }
}

/* ReLU6 (the activation of the MobileNetV2 family among the paper's models)
 * joined to the stash: y = (x <= 0) ? +0 : (x >= 6 ? 6 : x); a NaN fails both
 * comparisons and is kept.  Then Algorithm 1 on y. */
uint64_t oracle_relu6_fwd_compress(const void *pre_act, uint64_t n, int kind,
                                   void *y, uint32_t *bitmap, void *values,
                                   uint64_t *prefix)
{
    int elem_size = oracle_elem_size(kind);
    const unsigned char *src = (const unsigned char *)pre_act;
    unsigned char *yo = (unsigned char *)y;
    unsigned char *val = (unsigned char *)values;
    uint64_t words = (n + 31) / 32;
    uint64_t j = 0;
    unsigned char act[8];

    for (uint64_t w = 0; w < words; ++w) bitmap[w] = 0;

    for (uint64_t i = 0; i < n; ++i) {
        if (i % CHUNK_ELEMS == 0) prefix[i / CHUNK_ELEMS] = j;
        const unsigned char *e = src + i * (uint64_t)elem_size;
        int ge6, lt6;
        cmp_six(e, kind, &ge6, &lt6);
        if (le_zero(e, kind)) memset(act, 0, (size_t)elem_size);
        else if (ge6)         six_pattern(kind, act);
        else                  memcpy(act, e, (size_t)elem_size);
        if (yo) memcpy(yo + i * (uint64_t)elem_size, act, (size_t)elem_size);
        if (!all_bytes_zero(act, elem_size)) {
            memcpy(val + j * (uint64_t)elem_size, act, (size_t)elem_size);
            j += 1;
            bitmap[i >> 5] |= (uint32_t)1 << (i & 31);
        }
    }
    return j;
}

/* ReLU6 backward from the stash: the gradient passes where 0 < x < 6, i.e.
 * where the bit is set and the stashed activation is below 6 (a stashed 6 is a
 * saturated unit, a stashed NaN compares false); a select, as for ReLU.  Walks
 * the values with the single running counter of Algorithm 2. */
void oracle_relu6_bwd_from_stash(const uint32_t *bitmap, const void *values,
                                 uint64_t n, int kind, const void *grad_out,
                                 void *grad_in)
{
    int elem_size = oracle_elem_size(kind);
    const unsigned char *val = (const unsigned char *)values;
    const unsigned char *g = (const unsigned char *)grad_out;
    unsigned char *o = (unsigned char *)grad_in;
    uint64_t j = 0;
    for (uint64_t i = 0; i < n; ++i) {
        int pass = 0;
        if ((bitmap[i >> 5] >> (i & 31)) & 1u) {
            int ge6, lt6;
            cmp_six(val + j * (uint64_t)elem_size, kind, &ge6, &lt6);
            pass = lt6;
            j += 1;
        }
        if (pass) memmove(o + i * (uint64_t)elem_size, g + i * (uint64_t)elem_size, (size_t)elem_size);
        else      memset(o + i * (uint64_t)elem_size, 0, (size_t)elem_size);
    }
}

/* The ReLU gradient needs only the bitmap: a select, not a multiply, so that a
 * masked lane is +0 whatever the upstream gradient holds (-x, inf, NaN). */
void oracle_relu_bwd_from_bitmap(const uint32_t *bitmap, const void *grad_out,
                                 uint64_t n, int elem_size, void *grad_in)
{
    const unsigned char *g = (const unsigned char *)grad_out;
    unsigned char *o = (unsigned char *)grad_in;
    for (uint64_t i = 0; i < n; ++i) {
        if ((bitmap[i >> 5] >> (i & 31)) & 1u)
            memmove(o + i * (uint64_t)elem_size, g + i * (uint64_t)elem_size, (size_t)elem_size);
        else
            memset(o + i * (uint64_t)elem_size, 0, (size_t)elem_size);
    }
}

/* M_b = elem_size * nnz + n/8 (section 3.2), with whole 32-bit bitmap words and
 * the 8-byte-per-chunk prefix array this layout adds. */
uint64_t oracle_compressed_bytes(uint64_t n, uint64_t nnz, int elem_size)
{
    uint64_t words  = (n + 31) / 32;
    uint64_t chunks = (n + CHUNK_ELEMS - 1) / CHUNK_ELEMS;
    return 4 * words + nnz * (uint64_t)elem_size + 8 * chunks;
}

/* binary32 -> binary16, round to nearest, ties to even (IEEE 754 conversion).
 * Above the largest half (65504) by half a unit in the last place or more:
 * infinity.  At or below 2^-25: zero (2^-25 is the tie between 0 and the
 * smallest subnormal, and 0 is the even one).  A NaN becomes the one quiet
 * NaN 0x7FFF, sign and payload dropped (the reading taken for the narrowed
 * stash).  Works on the bit pattern; no floating-point operation involved. */
uint16_t oracle_float_to_half(uint32_t u)
{
    uint32_t sign = (u >> 16) & 0x8000u;
    uint32_t a    = u & 0x7FFFFFFFu;
    if (a > 0x7F800000u) return 0x7FFFu;
    if (a >= 0x477FF000u) return (uint16_t)(sign | 0x7C00u);     /* >= 65520 (and inf) */
    if (a <= 0x33000000u) return (uint16_t)sign;                 /* <= 2^-25 */
    uint32_t expo = a >> 23;
    uint32_t q, rem, half;
    if (expo < 113u) {
        /* below 2^-14: a half subnormal, q units of 2^-24.  With the hidden bit
         * the value is m * 2^(expo-150), i.e. m >> (126 - expo) units. */
        uint32_t m     = (a & 0x7FFFFFu) | 0x800000u;
        uint32_t shift = 126u - expo;                            /* 14 .. 24 */
        q    = m >> shift;
        rem  = m & ((1u << shift) - 1u);
        half = 1u << (shift - 1u);
    } else {
        /* normal half: rebias 127 -> 15, keep 10 mantissa bits, round on the 13 dropped */
        q    = ((expo - 112u) << 10) | ((a >> 13) & 0x3FFu);
        rem  = a & 0x1FFFu;
        half = 0x1000u;
    }
    if (rem > half || (rem == half && (q & 1u))) q += 1u;        /* a carry runs into the exponent as it should */
    return (uint16_t)(sign | q);
}

/* binary32 -> bfloat16 (the top 16 bits), round to nearest, ties to even; a
 * value that rounds past the largest finite bfloat16 becomes infinity by the
 * same carry; a NaN becomes 0x7FFF. */
uint16_t oracle_float_to_bfloat16(uint32_t u)
{
    if ((u & 0x7FFFFFFFu) > 0x7F800000u) return 0x7FFFu;
    uint32_t q = u >> 16, rem = u & 0xFFFFu;
    if (rem > 0x8000u || (rem == 0x8000u && (q & 1u))) q += 1u;
    return (uint16_t)q;
}

/* Down-cast on stash: the tensor is binary32, the stashed values are 16 bits
 * wide.  act = fused ? ((x <= tau) ? +0 : x) : x; bit i is set where the
 * binary32 pattern of act is not all-zero -- so bitmap, prefix and the count
 * are those of the full-precision stash -- and the value pushed is act
 * narrowed to to_kind (ORACLE_F16 or ORACLE_BF16), which may be a zero when
 * act underflows.  y (binary32, may be NULL) receives act.  Returns nnz. */
uint64_t oracle_narrow_compress(const void *x, uint64_t n, int to_kind, int fused, float tau,
                                void *y, uint32_t *bitmap, uint16_t *values, uint64_t *prefix)
{
    const unsigned char *src = (const unsigned char *)x;
    unsigned char *yo = (unsigned char *)y;
    uint64_t words = (n + 31) / 32;
    uint64_t j = 0;

    for (uint64_t w = 0; w < words; ++w) bitmap[w] = 0;

    for (uint64_t i = 0; i < n; ++i) {
        if (i % CHUNK_ELEMS == 0) prefix[i / CHUNK_ELEMS] = j;
        uint32_t u;
        memcpy(&u, src + 4 * i, 4);
        if (fused && le_tau(src + 4 * i, ORACLE_F32, tau)) u = 0;
        if (yo) memcpy(yo + 4 * i, &u, 4);
        if (u != 0) {
            values[j] = to_kind == ORACLE_F16 ? oracle_float_to_half(u) : oracle_float_to_bfloat16(u);
            j += 1;
            bitmap[i >> 5] |= (uint32_t)1 << (i & 31);
        }
    }
    return j;
}

/* Restoring a narrowed stash into a binary32 tensor: Algorithm 2 with each
 * 16-bit value widened on the way (binary16 -> binary32 and bfloat16 ->
 * binary32 are both exact, NaN payloads shift into the upper mantissa bits);
 * elements whose bit is clear are +0. */
void oracle_widen_decompress(const uint32_t *bitmap, const uint16_t *values, uint64_t n,
                             int from_kind, void *dense_f32)
{
    unsigned char *out = (unsigned char *)dense_f32;
    uint64_t j = 0;
    for (uint64_t i = 0; i < n; ++i) {
        uint32_t u = 0;
        if ((bitmap[i >> 5] >> (i & 31)) & 1u) {
            uint16_t h = values[j];
            j += 1;
            if (from_kind == ORACLE_F16) {
                float f = oracle_half_to_float(h);
                memcpy(&u, &f, 4);
            } else {
                u = (uint32_t)h << 16;
            }
        }
        memcpy(out + 4 * i, &u, 4);
    }
}

/* The element widened to binary64 for an ordering decision (exact for all four kinds). */
static double as_double(const unsigned char *e, int kind)
{
    switch (kind) {
    case ORACLE_F32: { float f; memcpy(&f, e, 4); return (double)f; }
    case ORACLE_F64: { double d; memcpy(&d, e, 8); return d; }
    case ORACLE_F16: { uint16_t h; memcpy(&h, e, 2); return (double)oracle_half_to_float(h); }
    default: {
        uint16_t h; memcpy(&h, e, 2);
        uint32_t u = (uint32_t)h << 16; float f; memcpy(&f, &u, 4);
        return (double)f;
    }
    }
}

/* 2x2 max pooling, stride 2, of `planes` images of height x width elements (both
 * even), row-major.  The window is visited in the order (0,0), (0,1), (1,0),
 * (1,1); a later element replaces the current maximum when it is greater or
 * when it is a NaN (so the first of equal maxima wins, and the last NaN wins):
 * the rule of the framework's own pooling kernels, which the codes must agree
 * with.  y (planes x height/2 x width/2) receives a raw copy of the winner,
 * codes (may be NULL) its position 2*dy + dx, two bits per output, sixteen
 * outputs per 32-bit word, output o in bits 2*(o%16).. of word o/16; unused
 * bits of the last word are 0. */
void oracle_maxpool2x2_fwd(const void *x, uint64_t planes, uint64_t height, uint64_t width,
                           int kind, void *y, uint32_t *codes)
{
    int es = oracle_elem_size(kind);
    const unsigned char *src = (const unsigned char *)x;
    unsigned char *dst = (unsigned char *)y;
    uint64_t ho = height / 2, wo = width / 2;
    uint64_t outputs = planes * ho * wo;
    if (codes)
        for (uint64_t w = 0; w < (outputs + 15) / 16; ++w) codes[w] = 0;
    uint64_t o = 0;
    for (uint64_t p = 0; p < planes; ++p)
        for (uint64_t r = 0; r < ho; ++r)
            for (uint64_t c = 0; c < wo; ++c, ++o) {
                uint64_t best_at = 0;
                double   best    = 0.0;
                unsigned best_k  = 0;
                for (unsigned k = 0; k < 4; ++k) {
                    uint64_t at = (p * height + 2 * r + (k >> 1)) * width + 2 * c + (k & 1);
                    double   v  = as_double(src + at * (uint64_t)es, kind);
                    if (k == 0 || v > best || v != v) {
                        best = v; best_at = at; best_k = k;
                    }
                }
                memcpy(dst + o * (uint64_t)es, src + best_at * (uint64_t)es, (size_t)es);
                if (codes) codes[o >> 4] |= (uint32_t)best_k << (2 * (o & 15));
            }
}

/* Its backward pass from the codes alone: the gradient of an output goes to the
 * window position its code names, the other three positions get +0. */
void oracle_maxpool2x2_bwd(const uint32_t *codes, const void *grad_out, uint64_t planes,
                           uint64_t height, uint64_t width, int elem_size, void *grad_in)
{
    const unsigned char *g = (const unsigned char *)grad_out;
    unsigned char *gi = (unsigned char *)grad_in;
    uint64_t ho = height / 2, wo = width / 2;
    memset(gi, 0, (size_t)(planes * height * width * (uint64_t)elem_size));
    uint64_t o = 0;
    for (uint64_t p = 0; p < planes; ++p)
        for (uint64_t r = 0; r < ho; ++r)
            for (uint64_t c = 0; c < wo; ++c, ++o) {
                unsigned k  = (codes[o >> 4] >> (2 * (o & 15))) & 3u;
                uint64_t at = (p * height + 2 * r + (k >> 1)) * width + 2 * c + (k & 1);
                memcpy(gi + at * (uint64_t)elem_size, g + o * (uint64_t)elem_size, (size_t)elem_size);
            }
}
