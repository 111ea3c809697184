/*
 * zccl_oracle.c -- TEST INFRASTRUCTURE, not the product.
 *
 * A plain, slow, single-threaded CPU statement of what the ZCCL hot path computes: the fZ-light
 * error-bounded lossy codec (Section 3.3), its chunk-indexed stream (Section 3.5.2, PIPE-fZ-light), the
 * reduce-scatter hop "decompress, add local data, recompress" (Section 3.1.2, Eq. 2) and the emulated ring
 * Allreduce / Allgather / Bcast (Sections 3.1.1, 3.5, 3.5.1).  It follows the algorithm's steps in the paper's
 * order; there is no blocking, fusion or reordering here.  It shares no code with the CUDA path and is used
 * only by tests, the smoke check and the benchmark's cpu_baseline / reference legs.
 *
 * Build: gcc -O2 -ffp-contract=off -fPIC -shared (no fast-math: every float operation below is one IEEE
 * binary32 operation, rounded to nearest even, with no fused multiply-add).
 *
 * Pin status (see the "not gpu" tests):
 *   quantiser + whole codec ........ pinned (closed form: round trip == pointwise quantiser; error bound)
 *   stream size / constant blocks .. pinned (closed form from brute-force code lengths; constant-array limit)
 *   byte layout .................... parity unpinned against the paper (the paper gives no byte layout);
 *                                    checked against hand-computed vectors of the layout stated below
 *   fused hop ...................... pinned by definition: compress(decompress(a) + b)
 *   ring Allreduce ................. pinned (on-grid inputs give the exact textbook sum; Eq. 2 hard bound)
 *   Allgather / Bcast .............. pinned (one compression: error <= bound; own chunk bit-identical)
 *
 * Stream layout (little endian; where the paper is silent the choice is stated):
 *   header, 32 bytes: u32 magic 'Z','C','L','1'; u32 version word 0x05000001 (version 1, dtype 0 = fp32,
 *                     log2 block = 5); u64 n; f32 eb_abs; f32 s (quantisation step); u32 T (elements per
 *                     tile); u32 nT = ceil(n / T)
 *   index, 4*nT bytes: u32 per tile = inclusive prefix sum of the tiles' blob sizes in 4-byte words
 *                     (the paper's per-chunk 4-byte sizes at the front of the buffer, already scanned)
 *   blobs: per tile  [i32 outlier = quantised first value]
 *                    [one code-length byte per 32-element block, zero padded to a multiple of 4 bytes]
 *                    [for every block with code length L > 0: u32 sign word (bit j = delta_j < 0), then
 *                     L bit-plane words, plane k holding bit k of |delta_j| in bit j]
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
#define ZO_W_PRECISION   1

#define ZO_EB_ABS 0
#define ZO_EB_REL 1

#define ZO_FLAG_CONSISTENT_OWNER 1u
/* reduce operation of the collective computation framework (Section 3.2: Sum, Average, Max, Min), bits 1..2 */
#define ZO_OP_MASK 6u
#define ZO_OP_SUM 0u
#define ZO_OP_MAX 2u
#define ZO_OP_MIN 4u
#define ZO_OP_AVG 6u   /* Sum on every hop; the collective divides the result by the number of ranks at the end */

#define ZO_MAGIC   0x314C435Au /* bytes 'Z','C','L','1' */
#define ZO_VERSION 0x05000001u
#define ZO_BLOCK   32u
#define ZO_HEADER  32u

/* ---------------------------------------------------------------- little-endian byte access */
static void put_u32(uint8_t *p, uint32_t v) { p[0] = (uint8_t)v; p[1] = (uint8_t)(v >> 8); p[2] = (uint8_t)(v >> 16); p[3] = (uint8_t)(v >> 24); }
static uint32_t get_u32(const uint8_t *p) { return (uint32_t)p[0] | ((uint32_t)p[1] << 8) | ((uint32_t)p[2] << 16) | ((uint32_t)p[3] << 24); }
static void put_u64(uint8_t *p, uint64_t v) { put_u32(p, (uint32_t)v); put_u32(p + 4, (uint32_t)(v >> 32)); }
static uint64_t get_u64(const uint8_t *p) { return (uint64_t)get_u32(p) | ((uint64_t)get_u32(p + 4) << 32); }
static void put_f32(uint8_t *p, float f) { uint32_t u; memcpy(&u, &f, 4); put_u32(p, u); }
static float get_f32(const uint8_t *p) { uint32_t u = get_u32(p); float f; memcpy(&f, &u, 4); return f; }

/* ---------------------------------------------------------------- bound resolution */

/* min and max of a float array (n >= 1). */
void zo_minmax(const float *x, size_t n, float *mn, float *mx)
{
    float lo = x[0], hi = x[0];
    for (size_t i = 1; i < n; ++i) { if (x[i] < lo) lo = x[i]; if (x[i] > hi) hi = x[i]; }
    *mn = lo; *mx = hi;
}

/* Error bound -> (eb_abs, s, r).  The paper quotes value-range-relative bounds ("REL", Tables 1-4) and says
 * only that quantisation is a multiplication (Section 3.3).  Reading: eb_abs = rel * (max - min); the step is
 * shrunk by 1 - 2^-6 so that fp32 rounding of x*r and q*s cannot push |x - x'| past eb_abs; r = 1/s by one
 * IEEE division. */
int zo_resolve_range(int eb_mode, float eb, float mn, float mx, float *eb_abs, float *s, float *r)
{
    if (!(eb > 0.0f) || !isfinite(eb)) return ZO_E_ARG;
    float ea;
    if (eb_mode == ZO_EB_REL) {
        float range = mx - mn;
        if (!(range > 0.0f) || !isfinite(range)) return ZO_E_DEGENERATE;
        ea = eb * range;
    } else if (eb_mode == ZO_EB_ABS) {
        ea = eb;
    } else return ZO_E_ARG;
    float ebq = ea * 0.984375f;
    float step = ebq * 2.0f;
    if (!(step > 0.0f) || !isfinite(step)) return ZO_E_DEGENERATE;
    float recip = 1.0f / step;
    if (!isfinite(recip)) return ZO_E_DEGENERATE;
    *eb_abs = ea; *s = step; *r = recip;
    return ZO_OK;
}

int zo_resolve(int eb_mode, float eb, const float *x, size_t n, float *eb_abs, float *s, float *r)
{
    float mn = 0.0f, mx = 0.0f;
    if (eb_mode == ZO_EB_REL) {
        if (n == 0) return ZO_E_DEGENERATE;
        zo_minmax(x, n, &mn, &mx);
    }
    return zo_resolve_range(eb_mode, eb, mn, mx, eb_abs, s, r);
}

/* ---------------------------------------------------------------- sizes */
static size_t pad4(size_t v) { return (v + 3u) & ~(size_t)3u; }

/* Worst-case stream size: every block at code length 31. */
size_t zo_compress_bound(size_t n, uint32_t T)
{
    if (T == 0) return 0;
    size_t nT = (n + T - 1) / T;
    size_t nB_full = T / ZO_BLOCK;
    size_t total = ZO_HEADER + 4 * nT;
    for (size_t t = 0; t < nT; ++t) {
        size_t len = (t + 1 == nT) ? n - t * (size_t)T : T;
        size_t nb = (t + 1 == nT) ? (len + ZO_BLOCK - 1) / ZO_BLOCK : nB_full;
        total += 4 + pad4(nb) + nb * 4 * 32;
    }
    return total;
}

/* ---------------------------------------------------------------- quantiser (Section 3.3: the multiplication) */

/* q_i = round-to-nearest-even( fl32(x_i * r) ).  Returns ZO_E_RANGE if any |x_i * r| >= 2^30 (then deltas of
 * neighbouring codes could not be held in 32 bits), else ZO_OK or ZO_W_PRECISION when some |q| > 2^15. */
int zo_quantise(const float *x, size_t n, float r, int32_t *q)
{
    int warn = 0;
    for (size_t i = 0; i < n; ++i) {
        float t = x[i] * r;
        if (!(fabsf(t) < 1073741824.0f)) return ZO_E_RANGE;
        int32_t qi = (int32_t)rintf(t);
        if (qi > 32768 || qi < -32768) warn = 1;
        q[i] = qi;
    }
    return warn ? ZO_W_PRECISION : ZO_OK;
}

static unsigned bitlen_u32(uint32_t v) { unsigned L = 0; while (v) { ++L; v >>= 1; } return L; }

/* ---------------------------------------------------------------- compress */
int zo_compress_core(const float *x, size_t n, float eb_abs, float s, float r, uint32_t T,
                     uint8_t *out, size_t cap, size_t *out_bytes)
{
    if (T == 0 || T % ZO_BLOCK != 0) return ZO_E_ARG;
    size_t nT = (n + T - 1) / T;
    if (nT > 0xFFFFFFFFu) return ZO_E_ARG;
    if (cap < ZO_HEADER + 4 * nT) return ZO_E_CAPACITY;

    put_u32(out + 0, ZO_MAGIC);
    put_u32(out + 4, ZO_VERSION);
    put_u64(out + 8, (uint64_t)n);
    put_f32(out + 16, eb_abs);
    put_f32(out + 20, s);
    put_u32(out + 24, T);
    put_u32(out + 28, (uint32_t)nT);

    int32_t *q = (int32_t *)malloc(sizeof(int32_t) * (size_t)T);
    int32_t *d = (int32_t *)malloc(sizeof(int32_t) * (size_t)T);
    if (!q || !d) { free(q); free(d); return ZO_E_ARG; }

    int warn = 0;
    size_t pos = ZO_HEADER + 4 * nT;   /* byte position of the next blob */
    uint64_t words = 0;                /* running blob size in 4-byte words */
    int rc = ZO_OK;

    for (size_t t = 0; t < nT; ++t) {
        size_t start = t * (size_t)T;
        size_t len = (n - start < T) ? n - start : T;
        size_t nb = (len + ZO_BLOCK - 1) / ZO_BLOCK;

        /* fused quantisation + 1-D Lorenzo prediction; the first code is the tile's outlier */
        int qrc = zo_quantise(x + start, len, r, q);
        if (qrc < 0) { rc = qrc; break; }
        if (qrc == ZO_W_PRECISION) warn = 1;
        d[0] = 0;
        for (size_t i = 1; i < len; ++i) d[i] = q[i] - q[i - 1];
        for (size_t i = len; i < nb * ZO_BLOCK; ++i) d[i] = 0;   /* tail lanes of the last block */

        if (pos + 4 + pad4(nb) > cap) { rc = ZO_E_CAPACITY; break; }
        put_u32(out + pos, (uint32_t)q[0]);
        uint8_t *Lbytes = out + pos + 4;
        memset(Lbytes, 0, pad4(nb));
        size_t p = pos + 4 + pad4(nb);

        for (size_t b = 0; b < nb; ++b) {
            const int32_t *db = d + b * ZO_BLOCK;
            uint32_t mx = 0;
            for (unsigned j = 0; j < ZO_BLOCK; ++j) {
                uint32_t a = db[j] < 0 ? (uint32_t)0 - (uint32_t)db[j] : (uint32_t)db[j];
                if (a > mx) mx = a;
            }
            unsigned L = bitlen_u32(mx);          /* code length: bits of the block's largest magnitude */
            Lbytes[b] = (uint8_t)L;
            if (L == 0) continue;                 /* constant block: the code-length byte is all that is stored */
            if (p + 4 * (1 + (size_t)L) > cap) { rc = ZO_E_CAPACITY; break; }
            uint32_t sign = 0;
            for (unsigned j = 0; j < ZO_BLOCK; ++j) if (db[j] < 0) sign |= (1u << j);
            put_u32(out + p, sign); p += 4;
            for (unsigned k = 0; k < L; ++k) {
                uint32_t plane = 0;
                for (unsigned j = 0; j < ZO_BLOCK; ++j) {
                    uint32_t a = db[j] < 0 ? (uint32_t)0 - (uint32_t)db[j] : (uint32_t)db[j];
                    if ((a >> k) & 1u) plane |= (1u << j);
                }
                put_u32(out + p, plane); p += 4;
            }
        }
        if (rc != ZO_OK) break;
        words += (p - pos) / 4;
        if (words > 0xFFFFFFFFu) { rc = ZO_E_CAPACITY; break; }
        put_u32(out + ZO_HEADER + 4 * t, (uint32_t)words);
        pos = p;
    }
    free(q); free(d);
    if (rc != ZO_OK) return rc;
    *out_bytes = pos;
    return warn ? ZO_W_PRECISION : ZO_OK;
}

int zo_compress(const float *x, size_t n, int eb_mode, float eb, uint32_t T,
                uint8_t *out, size_t cap, size_t *out_bytes)
{
    float eb_abs, s, r;
    int rc = zo_resolve(eb_mode, eb, x, n, &eb_abs, &s, &r);
    if (rc != ZO_OK) return rc;
    return zo_compress_core(x, n, eb_abs, s, r, T, out, cap, out_bytes);
}

/* ---------------------------------------------------------------- decompress */

/* Reads and validates the header.  Returns ZO_OK or ZO_E_BAD_STREAM. */
int zo_stream_info(const uint8_t *in, size_t in_bytes, uint64_t *n, float *eb_abs, float *s,
                   uint32_t *T, uint32_t *nT, size_t *total_bytes)
{
    if (in_bytes < ZO_HEADER) return ZO_E_BAD_STREAM;
    if (get_u32(in) != ZO_MAGIC || get_u32(in + 4) != ZO_VERSION) return ZO_E_BAD_STREAM;
    uint64_t nn = get_u64(in + 8);
    uint32_t TT = get_u32(in + 24), nTT = get_u32(in + 28);
    if (TT == 0 || TT % ZO_BLOCK != 0) return ZO_E_BAD_STREAM;
    if ((nn + TT - 1) / TT != nTT) return ZO_E_BAD_STREAM;
    if (in_bytes < ZO_HEADER + 4 * (size_t)nTT) return ZO_E_BAD_STREAM;
    size_t tot = ZO_HEADER + 4 * (size_t)nTT;
    if (nTT) tot += 4 * (size_t)get_u32(in + ZO_HEADER + 4 * ((size_t)nTT - 1));
    if (in_bytes < tot) return ZO_E_BAD_STREAM;
    float step = get_f32(in + 20);
    if (!(step > 0.0f) || !isfinite(step)) return ZO_E_BAD_STREAM;
    *n = nn; *eb_abs = get_f32(in + 16); *s = step; *T = TT; *nT = nTT; *total_bytes = tot;
    return ZO_OK;
}

/* Decodes the integer codes q (the state before the final multiplication); q_out may be NULL. */
int zo_decompress_codes(const uint8_t *in, size_t in_bytes, float *y, int32_t *q_out, size_t cap_elems, size_t *n_out)
{
    uint64_t n; float eb_abs, s; uint32_t T, nT; size_t total;
    int rc = zo_stream_info(in, in_bytes, &n, &eb_abs, &s, &T, &nT, &total);
    if (rc != ZO_OK) return rc;
    if (n > cap_elems) return ZO_E_CAPACITY;
    const uint8_t *idx = in + ZO_HEADER;
    size_t blob0 = ZO_HEADER + 4 * (size_t)nT;
    uint32_t prev_words = 0;
    for (size_t t = 0; t < nT; ++t) {
        uint32_t w = get_u32(idx + 4 * t);
        if (w < prev_words) return ZO_E_BAD_STREAM;
        size_t start = t * (size_t)T;
        size_t len = (n - start < T) ? (size_t)(n - start) : T;
        size_t nb = (len + ZO_BLOCK - 1) / ZO_BLOCK;
        size_t pos = blob0 + 4 * (size_t)prev_words;   /* chunk-starting location from the recorded sizes */
        size_t end = blob0 + 4 * (size_t)w;
        if (pos + 4 + pad4(nb) > end) return ZO_E_BAD_STREAM;
        int32_t acc = (int32_t)get_u32(in + pos);       /* outlier */
        const uint8_t *Lbytes = in + pos + 4;
        size_t p = pos + 4 + pad4(nb);
        for (size_t b = 0; b < nb; ++b) {
            unsigned L = Lbytes[b];
            if (L > 31) return ZO_E_BAD_STREAM;
            uint32_t sign = 0;
            const uint8_t *planes = NULL;
            if (L) {
                if (p + 4 * (1 + (size_t)L) > end) return ZO_E_BAD_STREAM;
                sign = get_u32(in + p);
                planes = in + p + 4;
                p += 4 * (1 + (size_t)L);
            }
            for (unsigned j = 0; j < ZO_BLOCK; ++j) {
                size_t i = b * ZO_BLOCK + j;
                if (i >= len) break;
                uint32_t a = 0;
                for (unsigned k = 0; k < L; ++k) a |= ((get_u32(planes + 4 * k) >> j) & 1u) << k;
                int32_t dlt = ((sign >> j) & 1u) ? (int32_t)((uint32_t)0 - a) : (int32_t)a;
                acc = (int32_t)((uint32_t)acc + (uint32_t)dlt);   /* undo Lorenzo: running sum from the outlier */
                if (q_out) q_out[start + i] = acc;
                if (y) y[start + i] = (float)acc * s;             /* one fp32 multiplication */
            }
        }
        if (p != end) return ZO_E_BAD_STREAM;
        prev_words = w;
    }
    if (n_out) *n_out = (size_t)n;
    return ZO_OK;
}

int zo_decompress(const uint8_t *in, size_t in_bytes, float *y, size_t cap_elems, size_t *n_out)
{
    return zo_decompress_codes(in, in_bytes, y, NULL, cap_elems, n_out);
}

/* ---------------------------------------------------------------- reduce-scatter hop (Section 3.1.2, Eq. 2) */

/* out_c = compress( decompress(in_c) (+) local ), written as exactly that composition; (+) is the addition unless
 * flags select Max or Min (the larger / the smaller of the two, the decoded operand kept when they compare equal).  Exactly one of `local`
 * (uncompressed fp32 chunk: the paper's form) and `local_c` (a second compressed chunk) is non-NULL.  The bound
 * and step are those of in_c's header (one bound for the whole collective).  raw_out, if given, receives the
 * fp32 sum y, or float(q(y))*s when ZO_FLAG_CONSISTENT_OWNER is set. */
int zo_drc(const uint8_t *in_c, size_t in_bytes, const float *local, const uint8_t *local_c, size_t local_c_bytes,
           size_t n_expected, uint8_t *out_c, size_t cap, size_t *out_bytes, float *raw_out, unsigned flags)
{
    if ((local == NULL) == (local_c == NULL)) return ZO_E_ARG;
    uint64_t n; float eb_abs, s; uint32_t T, nT; size_t total;
    int rc = zo_stream_info(in_c, in_bytes, &n, &eb_abs, &s, &T, &nT, &total);
    if (rc != ZO_OK) return rc;
    if (n != n_expected) return ZO_E_BAD_STREAM;
    float r = 1.0f / s;
    size_t m = (size_t)n;
    float *a = (float *)malloc(sizeof(float) * (m ? m : 1));
    float *b = NULL;
    if (!a) return ZO_E_ARG;
    rc = zo_decompress(in_c, in_bytes, a, m, NULL);
    if (rc != ZO_OK) { free(a); return rc; }
    if (local_c) {
        uint64_t n2; float e2, s2; uint32_t T2, nT2; size_t tot2;
        rc = zo_stream_info(local_c, local_c_bytes, &n2, &e2, &s2, &T2, &nT2, &tot2);
        if (rc == ZO_OK && (n2 != n || T2 != T || memcmp(&s2, &s, 4) != 0)) rc = ZO_E_BAD_STREAM;
        if (rc != ZO_OK) { free(a); return rc; }
        b = (float *)malloc(sizeof(float) * (m ? m : 1));
        if (!b) { free(a); return ZO_E_ARG; }
        rc = zo_decompress(local_c, local_c_bytes, b, m, NULL);
        if (rc != ZO_OK) { free(a); free(b); return rc; }
        local = b;
    }
    unsigned op = flags & ZO_OP_MASK;
    for (size_t i = 0; i < m; ++i) {   /* decoded partial on the left, one fp32 operation */
        if (op == ZO_OP_MAX) a[i] = (a[i] < local[i]) ? local[i] : a[i];
        else if (op == ZO_OP_MIN) a[i] = (local[i] < a[i]) ? local[i] : a[i];
        else a[i] = a[i] + local[i];
    }
    rc = zo_compress_core(a, m, eb_abs, s, r, T, out_c, cap, out_bytes);
    if (rc >= 0 && raw_out) {
        if (flags & ZO_FLAG_CONSISTENT_OWNER) {
            int rc2 = zo_decompress(out_c, *out_bytes, raw_out, m, NULL);
            if (rc2 != ZO_OK) rc = rc2;
        } else {
            memcpy(raw_out, a, sizeof(float) * m);
        }
    }
    free(a); free(b);
    return rc;
}

/* ---------------------------------------------------------------- emulated collectives: N ranks = N host arrays */

static void chunk_span(size_t n, int N, int c, size_t *off, size_t *len)
{
    size_t m = (n + (size_t)N - 1) / (size_t)N;
    size_t o = (size_t)c * m;
    if (o > n) o = n;
    size_t l = n - o < m ? n - o : m;
    *off = o; *len = l;
}

static int resolve_over_ranks(const float *const *send, int N, size_t n, int eb_mode, float eb,
                              float *eb_abs, float *s, float *r)
{
    float mn = 0.0f, mx = 0.0f;
    if (eb_mode == ZO_EB_REL) {
        if (n == 0) return ZO_E_DEGENERATE;
        zo_minmax(send[0], n, &mn, &mx);
        for (int k = 1; k < N; ++k) {
            float a, b; zo_minmax(send[k], n, &a, &b);
            if (a < mn) mn = a;
            if (b > mx) mx = b;
        }
    }
    return zo_resolve_range(eb_mode, eb, mn, mx, eb_abs, s, r);
}

/* Ring Allreduce (sum) = ring reduce-scatter in the collective computation framework followed by ring allgather
 * in the collective data movement framework (Section 3.5).  Chunk c of every rank's buffer is elements
 * [c*m, (c+1)*m), m = ceil(n/N).  Step 0: rank r compresses its chunk r.  Hop k = 0..N-2: rank r receives from
 * rank r-1 the stream of chunk (r-k-1) mod N, decodes it, adds its own uncompressed chunk and recompresses (Eq. 2:
 * N compressions for N ranks).  The last hop's recompression is the allgather's single compression; its owner,
 * rank r for chunk (r+1) mod N, keeps the uncompressed sum (ranks do not decompress what they compressed) unless
 * ZO_FLAG_CONSISTENT_OWNER asks for the dequantised value.  Then N-1 forwarding hops of compressed bytes and
 * one decompression of each foreign chunk.
 * hop_bytes (optional, N*N entries): hop_bytes[k*N + r] = compressed bytes rank r sent after step k
 * (k = 0 is the initial compression). */
int zo_sim_allreduce(const float *const *send, float *const *recv, int N, size_t n, int eb_mode, float eb,
                     unsigned flags, uint32_t T, size_t *hop_bytes)
{
    if (N < 1) return ZO_E_ARG;
    float eb_abs, s, r;
    int rc = resolve_over_ranks(send, N, n, eb_mode, eb, &eb_abs, &s, &r);
    if (rc != ZO_OK) return rc;
    size_t m = (n + (size_t)N - 1) / (size_t)N;
    size_t cap = zo_compress_bound(m, T);
    int warn = 0;
    /* cur[r]: the stream rank r holds and will send next; nxt[r]: what it produces this hop */
    uint8_t **cur = (uint8_t **)calloc((size_t)N, sizeof(uint8_t *));
    uint8_t **nxt = (uint8_t **)calloc((size_t)N, sizeof(uint8_t *));
    size_t *cur_b = (size_t *)calloc((size_t)N, sizeof(size_t));
    size_t *nxt_b = (size_t *)calloc((size_t)N, sizeof(size_t));
    for (int k = 0; k < N; ++k) { cur[k] = (uint8_t *)malloc(cap); nxt[k] = (uint8_t *)malloc(cap); }

    for (int rk = 0; rk < N && rc >= 0; ++rk) {
        size_t off, len; chunk_span(n, N, rk, &off, &len);
        rc = zo_compress_core(send[rk] + off, len, eb_abs, s, r, T, cur[rk], cap, &cur_b[rk]);
        if (rc == ZO_W_PRECISION) warn = 1;
        if (hop_bytes) hop_bytes[rk] = cur_b[rk];
    }
    if (N == 1 && rc >= 0) memcpy(recv[0], send[0], sizeof(float) * n);   /* nothing to reduce or move */

    for (int k = 0; k + 1 < N && rc >= 0; ++k) {
        for (int rk = 0; rk < N && rc >= 0; ++rk) {
            int from = (rk - 1 + N) % N;
            int c = ((rk - k - 1) % N + N) % N;
            size_t off, len; chunk_span(n, N, c, &off, &len);
            int last = (k == N - 2);
            rc = zo_drc(cur[from], cur_b[from], send[rk] + off, NULL, 0, len, nxt[rk], cap, &nxt_b[rk],
                        last ? recv[rk] + off : NULL, flags);
            if (rc == ZO_W_PRECISION) warn = 1;
            if (hop_bytes && rc >= 0) hop_bytes[(size_t)(k + 1) * (size_t)N + (size_t)rk] = nxt_b[rk];
        }
        for (int rk = 0; rk < N; ++rk) { uint8_t *tp = cur[rk]; cur[rk] = nxt[rk]; nxt[rk] = tp; size_t tb = cur_b[rk]; cur_b[rk] = nxt_b[rk]; nxt_b[rk] = tb; }
    }
    /* allgather stage: rank r now owns the stream of reduced chunk (r+1) mod N; forwarding hops only move
     * bytes, so every rank ends up holding every owner's stream; decode all but its own */
    for (int rk = 0; rk < N && rc >= 0 && N > 1; ++rk) {
        for (int owner = 0; owner < N && rc >= 0; ++owner) {
            if (owner == rk) continue;
            int c = (owner + 1) % N;
            size_t off, len; chunk_span(n, N, c, &off, &len);
            int rc2 = zo_decompress(cur[owner], cur_b[owner], recv[rk] + off, len, NULL);
            if (rc2 != ZO_OK) rc = rc2;
        }
    }
    if ((flags & ZO_OP_MASK) == ZO_OP_AVG && rc >= 0)   /* Average = Sum / N, one fp32 division per element */
        for (int rk = 0; rk < N; ++rk)
            for (size_t i = 0; i < n; ++i) recv[rk][i] = recv[rk][i] / (float)N;
    for (int k = 0; k < N; ++k) { free(cur[k]); free(nxt[k]); }
    free(cur); free(nxt); free(cur_b); free(nxt_b);
    if (rc < 0) return rc;
    return warn ? ZO_W_PRECISION : ZO_OK;
}

/* Ring Allgather in the collective data movement framework (Section 3.1.1): every rank compresses its
 * contribution once, compressed bytes circulate, each rank decompresses the N-1 foreign contributions and keeps
 * its own uncompressed.  recv[r] holds N*n elements.  sizes (optional, N entries) = compressed bytes per rank. */
int zo_sim_allgather(const float *const *send, float *const *recv, int N, size_t n, int eb_mode, float eb,
                     uint32_t T, size_t *sizes)
{
    if (N < 1) return ZO_E_ARG;
    float eb_abs, s, r;
    int rc = resolve_over_ranks(send, N, n, eb_mode, eb, &eb_abs, &s, &r);
    if (rc != ZO_OK) return rc;
    size_t cap = zo_compress_bound(n, T);
    int warn = 0;
    uint8_t **st = (uint8_t **)calloc((size_t)N, sizeof(uint8_t *));
    size_t *sb = (size_t *)calloc((size_t)N, sizeof(size_t));
    for (int k = 0; k < N; ++k) st[k] = (uint8_t *)malloc(cap);
    for (int rk = 0; rk < N && rc >= 0; ++rk) {
        rc = zo_compress_core(send[rk], n, eb_abs, s, r, T, st[rk], cap, &sb[rk]);
        if (rc == ZO_W_PRECISION) warn = 1;
        if (sizes) sizes[rk] = sb[rk];
    }
    for (int rk = 0; rk < N && rc >= 0; ++rk) {
        for (int src = 0; src < N && rc >= 0; ++src) {
            if (src == rk) { memcpy(recv[rk] + (size_t)src * n, send[rk], sizeof(float) * n); continue; }
            int rc2 = zo_decompress(st[src], sb[src], recv[rk] + (size_t)src * n, n, NULL);
            if (rc2 != ZO_OK) rc = rc2;
        }
    }
    for (int k = 0; k < N; ++k) free(st[k]);
    free(st); free(sb);
    if (rc < 0) return rc;
    return warn ? ZO_W_PRECISION : ZO_OK;
}

/* Broadcast in the data movement framework: the root compresses once, every sink decompresses that one stream
 * (tree forwarding moves bytes only). */
int zo_sim_bcast(const float *root, float *const *recv, int nsinks, size_t n, int eb_mode, float eb, uint32_t T,
                 size_t *stream_bytes)
{
    if (nsinks < 0) return ZO_E_ARG;
    size_t cap = zo_compress_bound(n, T);
    uint8_t *st = (uint8_t *)malloc(cap);
    size_t sb = 0;
    int rc = zo_compress(root, n, eb_mode, eb, T, st, cap, &sb);
    int warn = (rc == ZO_W_PRECISION);
    for (int k = 0; k < nsinks && rc >= 0; ++k) {
        int rc2 = zo_decompress(st, sb, recv[k], n, NULL);
        if (rc2 != ZO_OK) rc = rc2;
    }
    if (stream_bytes) *stream_bytes = sb;
    free(st);
    if (rc < 0) return rc;
    return warn ? ZO_W_PRECISION : ZO_OK;
}

/* Ring Reduce-scatter in the collective computation framework (Section 3.1.2; first stage of the Allreduce of
 * Section 3.1.3), as a collective of its own: rank r ends with chunk r of the element-wise sum, uncompressed.
 * Chunk c starts at rank c+1 (compressed there), travels c+1 -> c+2 -> ... -> c, and every receiver decompresses,
 * adds its own chunk c and, unless it is the last one, compresses the partial sum again: N-1 compressions per
 * chunk, the last rank keeps the sum it formed.  recv[r] holds the elements of chunk r.
 * hop_bytes (optional, (N-1)*N entries): hop_bytes[k*N + r] = compressed bytes rank r sent in step k. */
int zo_sim_reduce_scatter(const float *const *send, float *const *recv, int N, size_t n, int eb_mode, float eb,
                          uint32_t T, size_t *hop_bytes)
{
    if (N < 1) return ZO_E_ARG;
    float eb_abs, s, r;
    int rc = resolve_over_ranks(send, N, n, eb_mode, eb, &eb_abs, &s, &r);
    if (rc != ZO_OK) return rc;
    size_t m = (n + (size_t)N - 1) / (size_t)N;
    size_t cap = zo_compress_bound(m, T);
    int warn = 0;
    if (N == 1) { memcpy(recv[0], send[0], sizeof(float) * n); return ZO_OK; }
    uint8_t **cur = (uint8_t **)calloc((size_t)N, sizeof(uint8_t *));
    uint8_t **nxt = (uint8_t **)calloc((size_t)N, sizeof(uint8_t *));
    size_t *cur_b = (size_t *)calloc((size_t)N, sizeof(size_t));
    size_t *nxt_b = (size_t *)calloc((size_t)N, sizeof(size_t));
    for (int k = 0; k < N; ++k) { cur[k] = (uint8_t *)malloc(cap); nxt[k] = (uint8_t *)malloc(cap); }

    for (int rk = 0; rk < N && rc >= 0; ++rk) {          /* step 0: rank rk compresses chunk rk-1 */
        int c = (rk - 1 + N) % N;
        size_t off, len; chunk_span(n, N, c, &off, &len);
        rc = zo_compress_core(send[rk] + off, len, eb_abs, s, r, T, cur[rk], cap, &cur_b[rk]);
        if (rc == ZO_W_PRECISION) warn = 1;
        if (hop_bytes) hop_bytes[rk] = cur_b[rk];
    }
    for (int k = 0; k + 1 < N && rc >= 0; ++k) {           /* step k+1: rank rk receives chunk rk-k-2 from rk-1 */
        int last = (k == N - 2);
        for (int rk = 0; rk < N && rc >= 0; ++rk) {
            int from = (rk - 1 + N) % N;
            int c = ((rk - k - 2) % N + N) % N;
            size_t off, len; chunk_span(n, N, c, &off, &len);
            rc = zo_drc(cur[from], cur_b[from], send[rk] + off, NULL, 0, len, nxt[rk], cap, &nxt_b[rk],
                        last ? recv[rk] : NULL, 0u);
            if (rc == ZO_W_PRECISION) warn = 1;
            if (hop_bytes && rc >= 0 && !last) hop_bytes[(size_t)(k + 1) * (size_t)N + (size_t)rk] = nxt_b[rk];
        }
        for (int rk = 0; rk < N; ++rk) { uint8_t *tp = cur[rk]; cur[rk] = nxt[rk]; nxt[rk] = tp; size_t tb = cur_b[rk]; cur_b[rk] = nxt_b[rk]; nxt_b[rk] = tb; }
    }
    for (int k = 0; k < N; ++k) { free(cur[k]); free(nxt[k]); }
    free(cur); free(nxt); free(cur_b); free(nxt_b);
    if (rc < 0) return rc;
    return warn ? ZO_W_PRECISION : ZO_OK;
}

/* Scatter in the data movement framework over the binomial tree (Section 4.4): the root (rank 0) holds N chunks of
 * n elements, compresses chunks 1..N-1 once each, the tree forwards compressed bytes only (in the round with
 * distance d = the largest power of two below N, then d/2, ..., 1, every holder h hands the chunks h+d .. h+2d-1
 * to rank h+d), every rank decompresses its own chunk; the root keeps chunk 0 as it is.  recv[r] holds n elements.
 * sizes (optional, N entries; sizes[0] = 0): compressed bytes of each chunk.
 * round_bytes (optional, one entry per round, at most 32): bytes that cross the tree's links in that round. */
int zo_sim_scatter(const float *root, float *const *recv, int N, size_t n, int eb_mode, float eb, uint32_t T,
                   size_t *sizes, size_t *round_bytes)
{
    if (N < 1) return ZO_E_ARG;
    float eb_abs, s, r;
    int rc = zo_resolve(eb_mode, eb, root, (size_t)N * n, &eb_abs, &s, &r);
    if (rc != ZO_OK) return rc;
    size_t cap = zo_compress_bound(n, T);
    int warn = 0;
    uint8_t *st = (uint8_t *)malloc(cap);
    size_t *sb = (size_t *)calloc((size_t)N, sizeof(size_t));
    memcpy(recv[0], root, sizeof(float) * n);
    for (int c = 1; c < N && rc >= 0; ++c) {
        rc = zo_compress_core(root + (size_t)c * n, n, eb_abs, s, r, T, st, cap, &sb[c]);
        if (rc == ZO_W_PRECISION) warn = 1;
        if (rc >= 0) {
            int rc2 = zo_decompress(st, sb[c], recv[c], n, NULL);
            if (rc2 != ZO_OK) rc = rc2;
        }
    }
    if (sizes) for (int c = 0; c < N; ++c) sizes[c] = sb[c];
    if (round_bytes) {
        int d = 1, round = 0;
        while (2 * d < N) d *= 2;
        for (; d >= 1 && N > 1; d /= 2, ++round) {
            size_t moved = 0;
            for (int h = 0; h < N; h += 2 * d)              /* holders of this round */
                for (int c = h + d; c < h + 2 * d && c < N; ++c) moved += sb[c];
            round_bytes[round] = moved;
        }
    }
    free(st); free(sb);
    if (rc < 0) return rc;
    return warn ? ZO_W_PRECISION : ZO_OK;
}

/* Quality of a reconstruction y of x (Section 4.1: the paper reports NRMSE and PSNR next to the bit rate
 * 32 / ratio; the definitions are the usual ones): everything in fp64, elements taken in order.
 *   out[0] = max |x_i - y_i|          out[1] = MSE = mean (x_i - y_i)^2
 *   out[2] = NRMSE = sqrt(MSE) / (max x - min x)      out[3] = PSNR = 20 log10((max x - min x) / sqrt(MSE)) dB
 *   out[4] = min x                    out[5] = max x
 * A constant x has no range: NRMSE and PSNR are then NaN; an exact reconstruction has PSNR = +inf. */
int zo_quality(const float *x, const float *y, size_t n, double *out)
{
    if (n == 0) return ZO_E_ARG;
    double maxerr = 0.0, sumsq = 0.0, lo = (double)x[0], hi = (double)x[0];
    for (size_t i = 0; i < n; ++i) {
        double d = (double)x[i] - (double)y[i];
        double a = fabs(d);
        if (a > maxerr) maxerr = a;
        sumsq += d * d;
        if ((double)x[i] < lo) lo = (double)x[i];
        if ((double)x[i] > hi) hi = (double)x[i];
    }
    double mse = sumsq / (double)n;
    double range = hi - lo;
    out[0] = maxerr; out[1] = mse; out[4] = lo; out[5] = hi;
    if (range > 0.0) {
        out[2] = sqrt(mse) / range;
        out[3] = mse > 0.0 ? 20.0 * log10(range / sqrt(mse)) : (double)INFINITY;
    } else {
        out[2] = (double)NAN; out[3] = (double)NAN;
    }
    return ZO_OK;
}

/* Code-length statistics of a stream (Section 4.1, the table of compression ratios and percentages of constant
 * blocks: a block whose code length is 0 is a constant block and costs one byte).  hist[L], L = 0..31, receives the
 * number of 32-element blocks stored with code length L; hist[32] the number of blocks.  The walk is that of the
 * decompressor: chunk starts from the sizes at the front, code-length bytes behind each tile's outlier. */
int zo_stream_stats(const uint8_t *in, size_t in_bytes, uint64_t *hist)
{
    uint64_t n; float eb_abs, s; uint32_t T, nT; size_t total;
    int rc = zo_stream_info(in, in_bytes, &n, &eb_abs, &s, &T, &nT, &total);
    if (rc != ZO_OK) return rc;
    for (int k = 0; k <= 32; ++k) hist[k] = 0;
    size_t blob0 = ZO_HEADER + 4 * (size_t)nT;
    uint32_t prev_words = 0;
    for (size_t t = 0; t < nT; ++t) {
        uint32_t w = get_u32(in + ZO_HEADER + 4 * t);
        if (w < prev_words) return ZO_E_BAD_STREAM;
        size_t start = t * (size_t)T;
        size_t len = (n - start < T) ? (size_t)(n - start) : T;
        size_t nb = (len + ZO_BLOCK - 1) / ZO_BLOCK;
        size_t pos = blob0 + 4 * (size_t)prev_words;
        if (pos + 4 + pad4(nb) > blob0 + 4 * (size_t)w) return ZO_E_BAD_STREAM;
        for (size_t b = 0; b < nb; ++b) {
            unsigned L = in[pos + 4 + b];
            if (L > 31) return ZO_E_BAD_STREAM;
            hist[L] += 1;
            hist[32] += 1;
        }
        prev_words = w;
    }
    return ZO_OK;
}
