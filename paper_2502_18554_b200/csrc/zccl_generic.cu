// Codec for streams whose tile size is not the 4096 elements the tuned kernels are built around (Section 3.5.2
// cuts the data into chunks of 5120 points; the tile size is a header field of the stream).  Plain kernels, one CTA
// per tile and one warp per block of 32, with the arithmetic of the tuned kernels' integer route: q = rint(x * r) by
// one fp32 multiplication and one conversion, deltas inside the tile, code length = bit length of the largest
// magnitude of a block, sign word and bit planes by ballots.  Compression takes three launches (tile sizes, their
// prefix with header and index, the blobs), decompression one.  Any tile size that is a multiple of 32 between
// 1024 and 8192 elements.
#include "zccl_internal.h"

#include <cstdlib>

namespace zccl {
namespace {

constexpr unsigned kFull = 0xFFFFFFFFu;
constexpr int kGenMaxBlocks = kGenericMaxTile / kBlock;   // 256

__device__ __forceinline__ uint32_t bitlen(uint32_t v) { return 32u - (uint32_t)__clz((int)v); }

// The two value types.  Everything behind the quantisation works on 32-bit codes and is the same for both; what
// differs is one multiplication and one conversion on the way in (q = rint(x * r)), one conversion and one
// multiplication on the way out (x' = q * s), the data-type field of the version word, and header words 4..5
// (binary32: bound and step; binary64: the step as one binary64; the bound itself is not stored).
__device__ __forceinline__ float vmul(float a, float b) { return __fmul_rn(a, b); }
__device__ __forceinline__ double vmul(double a, double b) { return __dmul_rn(a, b); }
__device__ __forceinline__ int32_t vrint(float t) { return __float2int_rn(t); }
__device__ __forceinline__ int32_t vrint(double t) { return __double2int_rn(t); }
__device__ __forceinline__ float vabs(float t) { return fabsf(t); }
__device__ __forceinline__ double vabs(double t) { return fabs(t); }
__device__ __forceinline__ void from_code(int32_t q, float s, float* y) { *y = __fmul_rn(__int2float_rn(q), s); }
__device__ __forceinline__ void from_code(int32_t q, double s, double* y) { *y = __dmul_rn(__int2double_rn(q), s); }
template <class V> struct Bound;
template <> struct Bound<float> { using type = Params; static constexpr uint32_t version = kVersion; };
template <> struct Bound<double> { using type = ParamsF64; static constexpr uint32_t version = kVersionF64; };
__device__ __forceinline__ void header_step_words(const Params& p, uint32_t& w4, uint32_t& w5) { w4 = __float_as_uint(p.eb_abs); w5 = __float_as_uint(p.s); }
__device__ __forceinline__ void header_step_words(const ParamsF64& p, uint32_t& w4, uint32_t& w5)
{
    const unsigned long long b = (unsigned long long)__double_as_longlong(p.s);
    w4 = (uint32_t)b; w5 = (uint32_t)(b >> 32);
}
__device__ __forceinline__ float step_from_header(uint32_t w4, uint32_t w5, float) { (void)w4; return __uint_as_float(w5); }
__device__ __forceinline__ double step_from_header(uint32_t w4, uint32_t w5, double) { return __longlong_as_double((long long)(((unsigned long long)w5 << 32) | w4)); }

// Delta of element e of a tile (its code minus its predecessor's; 0 for the first element and for the padding
// lanes of a ragged last block, which repeat the last element).  `t_abs` receives |x * r| for the range checks.
template <class V>
__device__ __forceinline__ int32_t delta_at(const V* __restrict__ xt, uint32_t e, uint32_t last, V r, V& t_abs, int32_t& q_out)
{
    const uint32_t ec = e < last ? e : last;
    const uint32_t em = e ? e - 1 : 0;
    const uint32_t ep = em < last ? em : last;
    const V t = vmul(__ldg(xt + ec), r), tp = vmul(__ldg(xt + ep), r);
    t_abs = vabs(t);
    const int32_t q = vrint(t), qp = vrint(tp);
    q_out = q;
    return q - qp;
}

// Pass 1 (emit == 0): words of every tile's blob into sizes[].  Pass 3 (emit == 1): the blobs themselves, at the
// places the index (written by the scan in between) gives them.
template <class V>
__global__ void __launch_bounds__(256) generic_encode_kernel(const V* __restrict__ x, unsigned long long n, uint32_t T, uint32_t nT,
                                                             typename Bound<V>::type hp, const typename Bound<V>::type* dev_params,
                                                             uint32_t* __restrict__ sizes, uint32_t* __restrict__ out,
                                                             const uint32_t* __restrict__ go, int emit, Workspace ws)
{
    using P = typename Bound<V>::type;
    __shared__ uint32_t Ls[kGenMaxBlocks];
    __shared__ uint32_t offs[kGenMaxBlocks + 1];
    __shared__ uint32_t wsum[8];
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const P p = dev_params ? *dev_params : hp;
    if (!p.valid) return;
    if (emit && *go == 0) return;
    uint32_t status = 0;
    for (uint32_t t = blockIdx.x; t < nT; t += gridDim.x) {
        const unsigned long long start = (unsigned long long)t * T;
        const uint32_t len = (uint32_t)((n - start < (unsigned long long)T) ? (n - start) : (unsigned long long)T);
        const uint32_t nb = (len + kBlock - 1) / kBlock;
        const V* xt = x + start;
        V tmax = 0;
        uint32_t words = 0;
        for (uint32_t b = warp; b < nb; b += 8) {
            V ta; int32_t q;
            const int32_t d = delta_at(xt, 32u * b + lane, len - 1, p.r, ta, q);
            tmax = fmaxf(tmax, ta);
            const uint32_t L = bitlen(__reduce_or_sync(kFull, (uint32_t)(d < 0 ? -d : d)));
            if (lane == 0) Ls[b] = L;
            words += L ? L + 1 : 0;
        }
#pragma unroll
        for (int s = 16; s; s >>= 1) { const V o = __shfl_xor_sync(kFull, tmax, s); tmax = o > tmax ? o : tmax; }
        if (!(tmax < (V)1073741824.0)) status |= kStRange;
        else if (sizeof(V) == 4 && tmax > (V)32768.5) status |= kStPrecision;   // binary64 keeps its bound over the whole code range
        if (lane == 0) wsum[warp] = words;
        __syncthreads();
        if (!emit) {
            if (tid == 0) {
                uint32_t tot = 1 + ((nb + 3) >> 2);
                for (int w = 0; w < 8; ++w) tot += wsum[w];
                sizes[t] = tot;
            }
        } else {
            // offsets of the blocks' slots inside the blob: prefix of their sizes in block order
            if (warp == 0) {
                uint32_t carry = 1 + ((nb + 3) >> 2);
                for (uint32_t b0 = 0; b0 < nb; b0 += 32) {
                    const uint32_t b = b0 + lane;
                    const uint32_t sz = (b < nb && Ls[b]) ? Ls[b] + 1 : 0;
                    uint32_t inc = sz;
#pragma unroll
                    for (int s = 1; s < 32; s <<= 1) {
                        const uint32_t v = __shfl_up_sync(kFull, inc, s);
                        if (lane >= s) inc += v;
                    }
                    if (b < nb) offs[b] = carry + inc - sz;
                    carry += __shfl_sync(kFull, inc, 31);
                }
            }
            __syncthreads();
            uint32_t* blob = out + kHeaderWords + nT + (t ? __ldg(out + kHeaderWords + t - 1) : 0u);
            if (tid == 0) {
                V ta; int32_t q0;
                (void)delta_at(xt, 0, len - 1, p.r, ta, q0);
                blob[0] = (uint32_t)q0;                     // the tile's outlier: the code of its first element
            }
            for (uint32_t w = tid; w < ((nb + 3) >> 2); w += 256) {   // code-length bytes, zero padded to a word
                uint32_t word = 0;
                for (uint32_t k = 0; k < 4; ++k) if (4 * w + k < nb) word |= Ls[4 * w + k] << (8 * k);
                blob[1 + w] = word;
            }
            for (uint32_t b = warp; b < nb; b += 8) {
                const uint32_t L = Ls[b];
                V ta; int32_t q;
                const int32_t d = delta_at(xt, 32u * b + lane, len - 1, p.r, ta, q);   // warp-uniform trip count below
                if (L) {
                    const uint32_t a = (uint32_t)(d < 0 ? -d : d);
                    uint32_t* slot = blob + offs[b];
                    const uint32_t sg = __ballot_sync(kFull, d < 0);
                    if (lane == 0) slot[0] = sg;
                    for (uint32_t k = 0; k < L; ++k) {
                        const uint32_t pl = __ballot_sync(kFull, (a >> k) & 1u);
                        if (lane == 0) slot[1 + k] = pl;
                    }
                }
            }
        }
        __syncthreads();
    }
    if (!emit && status) atomicOr(ws.status, status);
}

// Pass 2: inclusive prefix of the tile sizes = the index; header; stream length; capacity check.  One CTA.
template <class V>
__global__ void __launch_bounds__(1024) generic_scan_kernel(const uint32_t* __restrict__ sizes, unsigned long long n, uint32_t T, uint32_t nT,
                                                            typename Bound<V>::type hp, const typename Bound<V>::type* dev_params, uint32_t* __restrict__ out,
                                                            unsigned long long out_cap, size_t* __restrict__ out_bytes,
                                                            uint32_t* __restrict__ go, Workspace ws)
{
    __shared__ unsigned long long wtot[32];
    __shared__ unsigned long long carry_s;
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const typename Bound<V>::type p = dev_params ? *dev_params : hp;
    if (!p.valid) {
        if (tid == 0) { *out_bytes = 0; *go = 0; }
        return;
    }
    // total first: nothing is written unless the whole stream fits
    unsigned long long mine = 0;
    for (uint32_t t = tid; t < nT; t += 1024) mine += sizes[t];
#pragma unroll
    for (int s = 16; s; s >>= 1) mine += __shfl_xor_sync(kFull, mine, s);
    if (lane == 0) wtot[warp] = mine;
    __syncthreads();
    unsigned long long total = 0;
    for (int w = 0; w < 32; ++w) total += wtot[w];
    const unsigned long long bytes = (unsigned long long)kHeaderBytes + 4ull * nT + 4ull * total;
    const bool fits = bytes <= out_cap && total <= 0xFFFFFFFFull;
    __syncthreads();
    if (tid == 0) {
        *go = fits ? 1u : 0u;
        *out_bytes = fits ? (size_t)bytes : 0;
        if (!fits) atomicOr(ws.status, kStCapacity);
        carry_s = 0;
    }
    if (!fits) return;
    if (tid == 0) {
        out[0] = kMagic; out[1] = Bound<V>::version;
        out[2] = (uint32_t)n; out[3] = (uint32_t)(n >> 32);
        uint32_t w4, w5;
        header_step_words(p, w4, w5);
        out[4] = w4; out[5] = w5;
        out[6] = T; out[7] = nT;
    }
    __syncthreads();
    for (uint32_t t0 = 0; t0 < nT; t0 += 1024) {
        const uint32_t t = t0 + tid;
        const unsigned long long v = t < nT ? sizes[t] : 0;
        unsigned long long inc = v;
#pragma unroll
        for (int s = 1; s < 32; s <<= 1) {
            const unsigned long long u = __shfl_up_sync(kFull, inc, s);
            if (lane >= s) inc += u;
        }
        if (lane == 31) wtot[warp] = inc;
        __syncthreads();
        unsigned long long before = carry_s;
        for (int w = 0; w < warp; ++w) before += wtot[w];
        if (t < nT) out[kHeaderWords + t] = (uint32_t)(before + inc);
        __syncthreads();
        if (tid == 1023) carry_s = before + inc;
        __syncthreads();
    }
}

// Decompression: one CTA per tile.  Code-length bytes -> slot offsets; every warp rebuilds the deltas of its blocks
// and their running sums inside the block; block totals are then chained through shared memory.
template <class V>
__global__ void __launch_bounds__(256) generic_decode_kernel(const uint32_t* __restrict__ in, unsigned long long cap_bytes, uint32_t T,
                                                             V* __restrict__ y, unsigned long long y_cap, Workspace ws)
{
    __shared__ uint32_t Ls[kGenMaxBlocks];
    __shared__ uint32_t offs[kGenMaxBlocks + 1];
    __shared__ int32_t btot[kGenMaxBlocks];
    __shared__ int32_t pre[kGenericMaxTile];
    __shared__ uint32_t bad_s;
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    // header (the tuned kernels' reader insists on their own tile size, so it is read here)
    bool ok = cap_bytes >= (unsigned long long)kHeaderBytes;
    unsigned long long n = 0;
    uint32_t nT = 0, total_w = 0;
    V s = 1;
    if (ok) {
        n = (unsigned long long)__ldg(in + 2) | ((unsigned long long)__ldg(in + 3) << 32);
        s = step_from_header(__ldg(in + 4), __ldg(in + 5), V());
        nT = __ldg(in + 7);
        ok = __ldg(in + 0) == kMagic && __ldg(in + 1) == Bound<V>::version && __ldg(in + 6) == T && (n + T - 1) / T == nT &&
             cap_bytes >= (unsigned long long)kHeaderBytes + 4ull * nT && s > (V)0 && isfinite(s);
    }
    if (ok && nT) {
        total_w = __ldg(in + kHeaderWords + nT - 1);
        ok = ((unsigned long long)kHeaderWords + nT + total_w) * 4ull <= cap_bytes;
    }
    if (!ok) { if (tid == 0 && blockIdx.x == 0) atomicOr(ws.status, kStBadStream); return; }
    if (n > y_cap) { if (tid == 0 && blockIdx.x == 0) atomicOr(ws.status, kStCapacity); return; }
    if (tid == 0) bad_s = 0;
    __syncthreads();
    const uint32_t* blob0 = in + kHeaderWords + nT;
    for (uint32_t t = blockIdx.x; t < nT; t += gridDim.x) {
        const unsigned long long start = (unsigned long long)t * T;
        const uint32_t len = (uint32_t)((n - start < (unsigned long long)T) ? (n - start) : (unsigned long long)T);
        const uint32_t nb = (len + kBlock - 1) / kBlock, lw = (nb + 3) >> 2;
        const uint32_t w_beg = t ? __ldg(in + kHeaderWords + t - 1) : 0u, w_end = __ldg(in + kHeaderWords + t);
        bool bad = w_end < w_beg || w_end > total_w || w_end - w_beg < 1 + lw;
        const uint32_t* blob = blob0 + w_beg;
        if (!bad) {
            for (uint32_t w = tid; w < lw; w += 256) {
                const uint32_t word = __ldg(blob + 1 + w);
                for (uint32_t k = 0; k < 4; ++k) {
                    const uint32_t L = (word >> (8 * k)) & 0xFFu;
                    if (4 * w + k < nb) { Ls[4 * w + k] = L; if (L > 31u) atomicOr(&bad_s, 1u); }
                }
            }
        }
        __syncthreads();
        bad = bad || bad_s != 0;
        if (!bad && warp == 0) {
            uint32_t carry = 1 + lw;
            for (uint32_t b0 = 0; b0 < nb; b0 += 32) {
                const uint32_t b = b0 + lane;
                const uint32_t sz = (b < nb && Ls[b]) ? Ls[b] + 1 : 0;
                uint32_t inc = sz;
#pragma unroll
                for (int sh = 1; sh < 32; sh <<= 1) {
                    const uint32_t v = __shfl_up_sync(kFull, inc, sh);
                    if (lane >= sh) inc += v;
                }
                if (b < nb) offs[b] = carry + inc - sz;
                carry += __shfl_sync(kFull, inc, 31);
            }
            if (lane == 0) { offs[nb] = carry; if (carry != w_end - w_beg) atomicOr(&bad_s, 1u); }   // the slots fill the blob exactly
        }
        __syncthreads();
        bad = bad || bad_s != 0;
        if (!bad) {
            for (uint32_t b = warp; b < nb; b += 8) {
                const uint32_t L = Ls[b];
                int32_t d = 0;
                if (L) {
                    const uint32_t* slot = blob + offs[b];
                    const uint32_t sg = __ldg(slot);
                    uint32_t a = 0;
                    for (uint32_t k = 0; k < L; ++k) a |= ((__ldg(slot + 1 + k) >> lane) & 1u) << k;
                    d = ((sg >> lane) & 1u) ? -(int32_t)a : (int32_t)a;
                }
#pragma unroll
                for (int sh = 1; sh < 32; sh <<= 1) {
                    const int32_t v = __shfl_up_sync(kFull, d, sh);
                    if (lane >= sh) d += v;
                }
                pre[32 * b + lane] = d;
                if (lane == 31) btot[b] = d;
            }
        }
        __syncthreads();
        if (!bad && warp == 0) {   // block totals -> code of the element before each block, from the outlier
            int32_t carry = (int32_t)__ldg(blob);
            for (uint32_t b0 = 0; b0 < nb; b0 += 32) {
                const uint32_t b = b0 + lane;
                const int32_t v = b < nb ? btot[b] : 0;
                int32_t inc = v;
#pragma unroll
                for (int sh = 1; sh < 32; sh <<= 1) {
                    const int32_t u = __shfl_up_sync(kFull, inc, sh);
                    if (lane >= sh) inc += u;
                }
                if (b < nb) btot[b] = carry + inc - v;
                carry += __shfl_sync(kFull, inc, 31);
            }
        }
        __syncthreads();
        if (!bad) {
            for (uint32_t e = tid; e < len; e += 256)
                from_code(btot[e >> 5] + pre[e], s, y + start + e);
        } else if (tid == 0) {
            atomicOr(ws.status, kStBadStream);
        }
        __syncthreads();
        if (tid == 0) bad_s = 0;
        __syncthreads();
    }
}

// Minimum and maximum of a binary64 array into two ordered 64-bit keys; the last CTA to get there turns them and the
// relative bound into the resolved block for binary64 (the reading of the binary32 path with the shrink 1 - 2^-20,
// which keeps |x - x'| <= eb_abs over the whole code range) and re-arms the keys.
__device__ __forceinline__ unsigned long long d2key(double v)
{
    const unsigned long long b = (unsigned long long)__double_as_longlong(v);
    return (b >> 63) ? ~b : (b | 0x8000000000000000ull);
}
__device__ __forceinline__ double key2d(unsigned long long k)
{
    return __longlong_as_double((long long)((k >> 63) ? (k & 0x7FFFFFFFFFFFFFFFull) : ~k));
}
__device__ void resolve_f64(double ea, bool range_ok, const Workspace& ws)
{
    ParamsF64 p;
    p.valid = range_ok ? 1 : 0;
    const double ebq = __dmul_rn(ea, 1.0 - 9.5367431640625e-07);   // 1 - 2^-20
    const double s = __dmul_rn(ebq, 2.0);
    if (!(s > 0.0) || !isfinite(s)) p.valid = 0;
    const double r = __ddiv_rn(1.0, s);
    if (!isfinite(r)) p.valid = 0;
    p.eb_abs = ea; p.s = s; p.r = r;
    *ws.params64 = p;
    if (!p.valid) atomicOr(ws.status, kStDegenerate);
}
__global__ void __launch_bounds__(512, 2) range_f64_kernel(const double* __restrict__ x, unsigned long long n, double eb, Workspace ws)
{
    double lo = __longlong_as_double(0x7FF0000000000000ll), hi = __longlong_as_double((long long)0xFFF0000000000000ull);
    auto take = [&](double v) { lo = v < lo ? v : lo; hi = v > hi ? v : hi; };
    const unsigned long long tid = (unsigned long long)blockIdx.x * blockDim.x + threadIdx.x;
    const unsigned long long nthreads = (unsigned long long)gridDim.x * blockDim.x;
    // peel to a 16-byte boundary, then 128-bit loads, eight of them in flight per thread
    unsigned long long head = ((uintptr_t)x & 15u) ? 1u : 0u;
    if (head > n) head = n;
    if (tid < head) take(x[tid]);
    const unsigned long long nvec = (n - head) >> 1;
    const double2* xv = reinterpret_cast<const double2*>(x + head);
    unsigned long long i = tid;
    constexpr int kInFlight = 8;
    for (; i + (kInFlight - 1) * nthreads < nvec; i += kInFlight * nthreads) {
        double2 v[kInFlight];
#pragma unroll
        for (int k = 0; k < kInFlight; ++k) v[k] = __ldcs(xv + i + k * nthreads);
#pragma unroll
        for (int k = 0; k < kInFlight; ++k) { take(v[k].x); take(v[k].y); }
    }
    for (; i < nvec; i += nthreads) {
        const double2 v = __ldg(xv + i);
        take(v.x); take(v.y);
    }
    const unsigned long long tail0 = head + (nvec << 1);
    if (tail0 + tid < n) take(x[tail0 + tid]);
#pragma unroll
    for (int s = 16; s; s >>= 1) {
        const double a = __shfl_xor_sync(kFull, lo, s), b = __shfl_xor_sync(kFull, hi, s);
        lo = a < lo ? a : lo;
        hi = b > hi ? b : hi;
    }
    // one pair of keys per CTA (an atomic on one address costs about 1.5 ns, whoever issues it: large CTAs, few of them)
    __shared__ uint32_t last_s;
    __shared__ double s_lo[32], s_hi[32];
    if ((threadIdx.x & 31) == 0) { s_lo[threadIdx.x >> 5] = lo; s_hi[threadIdx.x >> 5] = hi; }
    __syncthreads();
    if (threadIdx.x == 0) {
        for (unsigned w = 1; w < (blockDim.x >> 5); ++w) { lo = s_lo[w] < lo ? s_lo[w] : lo; hi = s_hi[w] > hi ? s_hi[w] : hi; }
        if (lo <= hi) { atomicMin(ws.minmax64 + 0, d2key(lo)); atomicMax(ws.minmax64 + 1, d2key(hi)); }
        __threadfence();
        last_s = atomicAdd(ws.done, 1u) == gridDim.x - 1 ? 1u : 0u;
    }
    __syncthreads();
    if (last_s && threadIdx.x == 0) {
        __threadfence();
        *ws.done = 0;
        const unsigned long long kmin = *reinterpret_cast<volatile unsigned long long*>(ws.minmax64 + 0);
        const unsigned long long kmax = *reinterpret_cast<volatile unsigned long long*>(ws.minmax64 + 1);
        double range = 0.0;
        if (kmin <= kmax) range = __dsub_rn(key2d(kmax), key2d(kmin));
        ws.minmax64[0] = 0xFFFFFFFFFFFFFFFFull;
        ws.minmax64[1] = 0ull;
        resolve_f64(__dmul_rn(eb, range), range > 0.0 && isfinite(range), ws);
    }
}

}  // namespace

template <class V>
static cudaError_t generic_encode(const V* x, unsigned long long n, uint32_t T, typename Bound<V>::type hp, const typename Bound<V>::type* dev_params,
                                  uint32_t* sizes, uint32_t* go, uint32_t* out, unsigned long long out_cap, size_t* out_bytes,
                                  const Workspace& ws, int sm_count, cudaStream_t st)
{
    const uint32_t nT = (uint32_t)((n + T - 1) / T);
    const unsigned grid = nT < (unsigned)sm_count * 4u ? (nT ? nT : 1u) : (unsigned)sm_count * 4u;
    count_launches(3);
    generic_encode_kernel<V><<<grid, 256, 0, st>>>(x, n, T, nT, hp, dev_params, sizes, out, go, 0, ws);
    generic_scan_kernel<V><<<1, 1024, 0, st>>>(sizes, n, T, nT, hp, dev_params, out, out_cap, out_bytes, go, ws);
    generic_encode_kernel<V><<<grid, 256, 0, st>>>(x, n, T, nT, hp, dev_params, sizes, out, go, 1, ws);
    return cudaGetLastError();
}
template <class V>
static cudaError_t generic_decode(const uint32_t* in, unsigned long long cap_bytes, uint32_t T, V* y, unsigned long long y_cap, const Workspace& ws,
                                  int sm_count, cudaStream_t st)
{
    const unsigned long long nT = (y_cap + T - 1) / T;
    const unsigned cap = (unsigned)sm_count * 4u;
    const unsigned grid = nT < cap ? (unsigned)(nT ? nT : 1) : cap;
    count_launches(1);
    generic_decode_kernel<V><<<grid, 256, 0, st>>>(in, cap_bytes, T, y, y_cap, ws);
    return cudaGetLastError();
}

// ZCCL_PLAIN=1 in the environment keeps other tile sizes and binary64 on the plain kernels of this file (for comparison).
static bool plain_forced()
{
    static const bool forced = [] { const char* v = getenv("ZCCL_PLAIN"); return v && v[0] == '1'; }();
    return forced;
}

cudaError_t launch_generic_encode(const float* x, unsigned long long n, uint32_t T, Params hp, bool device_params, uint32_t* sizes,
                                  uint32_t* go, uint32_t* out, unsigned long long out_cap, size_t* out_bytes, const Workspace& ws,
                                  int sm_count, cudaStream_t st)
{
    if (tiled_lanes_fit(n, T, ws) && !plain_forced()) {
        count_launches(2);
        return launch_encode_tiled_lanes(x, n, T, hp, device_params, out, out_cap, out_bytes, ws, sm_count, st);
    }
    return generic_encode<float>(x, n, T, hp, device_params ? ws.params : nullptr, sizes, go, out, out_cap, out_bytes, ws, sm_count, st);
}

cudaError_t launch_generic_decode(const uint32_t* in, unsigned long long cap_bytes, uint32_t T, float* y, unsigned long long y_cap,
                                  const Workspace& ws, int sm_count, cudaStream_t st)
{
    if (!plain_forced()) {
        count_launches(1);
        return launch_decode_tiled_lanes(in, cap_bytes, T, y, y_cap, ws, sm_count, st);
    }
    return generic_decode<float>(in, cap_bytes, T, y, y_cap, ws, sm_count, st);
}

cudaError_t launch_encode_f64(const double* x, unsigned long long n, ParamsF64 hp, bool device_params, uint32_t* sizes, uint32_t* go,
                              uint32_t* out, unsigned long long out_cap, size_t* out_bytes, const Workspace& ws, int sm_count, cudaStream_t st)
{
    if (ws.slots && (n + kTile - 1) / kTile <= ws.max_tiles && !plain_forced()) {
        count_launches(2);
        return launch_encode_f64_lanes(x, n, hp, device_params, out, out_cap, out_bytes, ws, sm_count, st);
    }
    return generic_encode<double>(x, n, (uint32_t)kTile, hp, device_params ? ws.params64 : nullptr, sizes, go, out, out_cap, out_bytes, ws,
                                  sm_count, st);
}

cudaError_t launch_decode_f64(const uint32_t* in, unsigned long long cap_bytes, double* y, unsigned long long y_cap, const Workspace& ws,
                              int sm_count, cudaStream_t st)
{
    if (!plain_forced()) {
        count_launches(1);
        return launch_decode_f64_lanes(in, cap_bytes, y, y_cap, ws, sm_count, st);
    }
    return generic_decode<double>(in, cap_bytes, (uint32_t)kTile, y, y_cap, ws, sm_count, st);
}

cudaError_t launch_range_f64(const double* x, unsigned long long n, double eb, const Workspace& ws, int sm_count, cudaStream_t st)
{
    const unsigned long long want = (n / 2 + 511) / 512;
    const unsigned cap = (unsigned)sm_count * 2u;
    count_launches(1);
    range_f64_kernel<<<(unsigned)(want < cap ? (want ? want : 1) : cap), 512, 0, st>>>(x, n, eb, ws);
    return cudaGetLastError();
}

}  // namespace zccl
