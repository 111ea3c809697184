/*
 * zccl_oracle_f64.c -- TEST INFRASTRUCTURE, not the product.
 *
 * The fZ-light codec of zccl_oracle.c for binary64 input, written out in full once more (plain, slow, one thread,
 * the algorithm's steps in the paper's order: Section 3.3 multiplication and rounding, 1-D Lorenzo prediction,
 * per-block code length, fixed-length bit planes; Section 3.5.2 chunk sizes at the front).  The paper states the
 * method for floating-point data without tying it to a width; everything after the quantisation works on 32-bit
 * integer codes and is the same as for binary32.  Used only by tests and the benchmark's CPU legs.
 *
 * Readings for binary64 (where the paper is silent):
 *   bound     eb_abs is a binary64 number; a value-range-relative bound is eb_abs = fl64(eb * fl64(max - min))
 *   step      eb_q = fl64(eb_abs * (1 - 2^-20)), s = 2 * eb_q (exact), r = fl64(1 / s)
 *   codes     t = fl64(x * r); range error unless |t| < 2^30; q = t rounded to the nearest integer, ties to even
 *   values    x' = fl64((double)q * s)
 *   The shrink by 2^-20 pays for the three roundings (of r, of x * r, of q * s: together below 3 * 2^-53 * |x|, and
 *   |x| < 2^30 * s): |x - x'| <= eb_q * (1 + 3 * 2^-22) < eb_abs for EVERY code in range, so there is no
 *   precision warning for this width.
 *
 * Stream layout: that of zccl_oracle.c with the data-type field of the version word set (0x05000101: version 1,
 * dtype 1 = binary64, log2 block = 5) and header bytes 16..23 holding the step s as one binary64 (binary32
 * streams keep eb_abs and s there as two binary32 numbers).  Index and blobs are identical.
 *
 * Pin status: quantiser and round trip pinned (closed form in numpy binary64; error bound in exact rational
 * arithmetic on adversarial values); byte layout checked against hand-computed vectors (the paper gives none).
 *
 * Build: gcc -O2 -ffp-contract=off -fPIC -shared, together with zccl_oracle.c.
 */
#include <stddef.h>
#include <stdint.h>
#include <string.h>
#include <stdlib.h>
#include <math.h>

#define ZO_OK            0
#define ZO_E_ARG        -1
#define ZO_E_CAPACITY   -3
#define ZO_E_RANGE      -4
#define ZO_E_BAD_STREAM -5
#define ZO_E_DEGENERATE -7
#define ZO_EB_ABS 0
#define ZO_EB_REL 1

#define ZO_MAGIC       0x314C435Au
#define ZO_VERSION_F64 0x05000101u
#define ZO_BLOCK       32u
#define ZO_HEADER      32u

static void put32(uint8_t *p, uint32_t v) { p[0] = (uint8_t)v; p[1] = (uint8_t)(v >> 8); p[2] = (uint8_t)(v >> 16); p[3] = (uint8_t)(v >> 24); }
static uint32_t get32(const uint8_t *p) { return (uint32_t)p[0] | ((uint32_t)p[1] << 8) | ((uint32_t)p[2] << 16) | ((uint32_t)p[3] << 24); }
static void put64(uint8_t *p, uint64_t v) { put32(p, (uint32_t)v); put32(p + 4, (uint32_t)(v >> 32)); }
static uint64_t get64(const uint8_t *p) { return (uint64_t)get32(p) | ((uint64_t)get32(p + 4) << 32); }
static size_t pad4w(size_t v) { return (v + 3u) & ~(size_t)3u; }
static unsigned bitlen32(uint32_t v) { unsigned L = 0; while (v) { ++L; v >>= 1; } return L; }

/* eb -> (eb_abs, s, r) in binary64; mn, mx are looked at for a relative bound only. */
int zo_resolve_f64(int eb_mode, double eb, double mn, double mx, double *eb_abs, double *s, double *r)
{
    if (!(eb > 0.0) || !isfinite(eb)) return ZO_E_ARG;
    volatile double ea = eb;
    if (eb_mode == ZO_EB_REL) {
        volatile double range = mx - mn;
        if (!(mn <= mx) || !(range > 0.0) || !isfinite(range)) return ZO_E_DEGENERATE;
        ea = eb * range;
    } else if (eb_mode != ZO_EB_ABS) return ZO_E_ARG;
    volatile double ebq = ea * (1.0 - 9.5367431640625e-07);   /* 1 - 2^-20, exact */
    volatile double step = ebq * 2.0;
    if (!(step > 0.0) || !isfinite(step)) return ZO_E_DEGENERATE;
    volatile double rec = 1.0 / step;
    if (!isfinite(rec)) return ZO_E_DEGENERATE;
    *eb_abs = ea; *s = step; *r = rec;
    return ZO_OK;
}

/* q_i = nearest integer (ties to even) of fl64(x_i * r); ZO_E_RANGE if some |x_i * r| >= 2^30. */
int zo_quantise_f64(const double *x, size_t n, double r, int32_t *q)
{
    for (size_t i = 0; i < n; ++i) {
        volatile double t = x[i] * r;
        if (!(fabs(t) < 1073741824.0)) return ZO_E_RANGE;
        q[i] = (int32_t)rint(t);
    }
    return ZO_OK;
}

int zo_compress_f64(const double *x, size_t n, int eb_mode, double eb, uint32_t T, uint8_t *out, size_t cap, size_t *out_bytes)
{
    if (T == 0 || T % ZO_BLOCK != 0) return ZO_E_ARG;
    double mn = 0.0, mx = 0.0;
    if (eb_mode == ZO_EB_REL) {
        if (n == 0) return ZO_E_DEGENERATE;
        mn = mx = x[0];
        for (size_t i = 1; i < n; ++i) { if (x[i] < mn) mn = x[i]; if (x[i] > mx) mx = x[i]; }
    }
    double eb_abs, s, r;
    int rc = zo_resolve_f64(eb_mode, eb, mn, mx, &eb_abs, &s, &r);
    if (rc != ZO_OK) return rc;
    size_t nT = (n + T - 1) / T;
    if (nT > 0xFFFFFFFFu) return ZO_E_ARG;
    if (cap < ZO_HEADER + 4 * nT) return ZO_E_CAPACITY;

    put32(out + 0, ZO_MAGIC);
    put32(out + 4, ZO_VERSION_F64);
    put64(out + 8, (uint64_t)n);
    uint64_t sbits; memcpy(&sbits, &s, 8);
    put64(out + 16, sbits);
    put32(out + 24, T);
    put32(out + 28, (uint32_t)nT);

    int32_t *q = (int32_t *)malloc(sizeof(int32_t) * (size_t)T);
    int32_t *d = (int32_t *)malloc(sizeof(int32_t) * (size_t)T);
    if (!q || !d) { free(q); free(d); return ZO_E_ARG; }
    size_t pos = ZO_HEADER + 4 * nT;
    uint64_t words = 0;
    for (size_t t = 0; t < nT && rc == ZO_OK; ++t) {
        size_t start = t * (size_t)T;
        size_t len = (n - start < T) ? n - start : T;
        size_t nb = (len + ZO_BLOCK - 1) / ZO_BLOCK;
        rc = zo_quantise_f64(x + start, len, r, q);
        if (rc != ZO_OK) break;
        /* 1-D Lorenzo prediction inside the tile; the first code is kept whole (the tile's outlier) */
        d[0] = 0;
        for (size_t i = 1; i < len; ++i) d[i] = q[i] - q[i - 1];
        for (size_t i = len; i < nb * ZO_BLOCK; ++i) d[i] = 0;
        if (pos + 4 + pad4w(nb) > cap) { rc = ZO_E_CAPACITY; break; }
        put32(out + pos, (uint32_t)q[0]);
        uint8_t *Lbytes = out + pos + 4;
        memset(Lbytes, 0, pad4w(nb));
        size_t p = pos + 4 + pad4w(nb);
        for (size_t b = 0; b < nb; ++b) {
            const int32_t *db = d + b * ZO_BLOCK;
            uint32_t mag[32], largest = 0, sign = 0;
            for (unsigned j = 0; j < ZO_BLOCK; ++j) {
                mag[j] = db[j] < 0 ? (uint32_t)0 - (uint32_t)db[j] : (uint32_t)db[j];
                if (mag[j] > largest) largest = mag[j];
                if (db[j] < 0) sign |= 1u << j;
            }
            unsigned L = bitlen32(largest);
            Lbytes[b] = (uint8_t)L;
            if (L == 0) continue;
            if (p + 4 * (1 + (size_t)L) > cap) { rc = ZO_E_CAPACITY; break; }
            put32(out + p, sign); p += 4;
            for (unsigned k = 0; k < L; ++k) {
                uint32_t plane = 0;
                for (unsigned j = 0; j < ZO_BLOCK; ++j) plane |= ((mag[j] >> k) & 1u) << j;
                put32(out + p, plane); p += 4;
            }
        }
        if (rc != ZO_OK) break;
        words += (p - pos) / 4;
        if (words > 0xFFFFFFFFu) { rc = ZO_E_CAPACITY; break; }
        put32(out + ZO_HEADER + 4 * t, (uint32_t)words);
        pos = p;
    }
    free(q); free(d);
    if (rc != ZO_OK) return rc;
    *out_bytes = pos;
    return ZO_OK;
}

/* y (and, if q_out is not NULL, the integer codes) from a binary64 stream. */
int zo_decompress_f64(const uint8_t *in, size_t in_bytes, double *y, int32_t *q_out, size_t cap_elems, size_t *n_out)
{
    if (in_bytes < ZO_HEADER) return ZO_E_BAD_STREAM;
    if (get32(in) != ZO_MAGIC || get32(in + 4) != ZO_VERSION_F64) return ZO_E_BAD_STREAM;
    uint64_t n = get64(in + 8);
    uint64_t sbits = get64(in + 16);
    double s; memcpy(&s, &sbits, 8);
    uint32_t T = get32(in + 24), nT = get32(in + 28);
    if (T == 0 || T % ZO_BLOCK != 0 || (n + T - 1) / T != nT) return ZO_E_BAD_STREAM;
    if (!(s > 0.0) || !isfinite(s)) return ZO_E_BAD_STREAM;
    if (in_bytes < ZO_HEADER + 4 * (size_t)nT) return ZO_E_BAD_STREAM;
    if (nT && in_bytes < ZO_HEADER + 4 * (size_t)nT + 4 * (size_t)get32(in + ZO_HEADER + 4 * ((size_t)nT - 1))) return ZO_E_BAD_STREAM;
    if (n > cap_elems) return ZO_E_CAPACITY;
    size_t blob0 = ZO_HEADER + 4 * (size_t)nT;
    uint32_t prev = 0;
    for (size_t t = 0; t < nT; ++t) {
        uint32_t w = get32(in + ZO_HEADER + 4 * t);
        if (w < prev) return ZO_E_BAD_STREAM;
        size_t start = t * (size_t)T;
        size_t len = (n - start < T) ? (size_t)(n - start) : T;
        size_t nb = (len + ZO_BLOCK - 1) / ZO_BLOCK;
        size_t pos = blob0 + 4 * (size_t)prev, end = blob0 + 4 * (size_t)w;
        if (pos + 4 + pad4w(nb) > end) return ZO_E_BAD_STREAM;
        int32_t acc = (int32_t)get32(in + pos);
        const uint8_t *Lbytes = in + pos + 4;
        size_t p = pos + 4 + pad4w(nb);
        for (size_t b = 0; b < nb; ++b) {
            unsigned L = Lbytes[b];
            if (L > 31) return ZO_E_BAD_STREAM;
            uint32_t sign = 0;
            const uint8_t *planes = NULL;
            if (L) {
                if (p + 4 * (1 + (size_t)L) > end) return ZO_E_BAD_STREAM;
                sign = get32(in + p);
                planes = in + p + 4;
                p += 4 * (1 + (size_t)L);
            }
            for (unsigned j = 0; j < ZO_BLOCK; ++j) {
                size_t i = b * ZO_BLOCK + j;
                if (i >= len) break;
                uint32_t a = 0;
                for (unsigned k = 0; k < L; ++k) a |= ((get32(planes + 4 * k) >> j) & 1u) << k;
                int32_t dlt = ((sign >> j) & 1u) ? (int32_t)((uint32_t)0 - a) : (int32_t)a;
                acc = (int32_t)((uint32_t)acc + (uint32_t)dlt);
                if (q_out) q_out[start + i] = acc;
                if (y) { volatile double v = (double)acc * s; y[start + i] = v; }
            }
        }
        if (p != end) return ZO_E_BAD_STREAM;
        prev = w;
    }
    if (n_out) *n_out = (size_t)n;
    return ZO_OK;
}
