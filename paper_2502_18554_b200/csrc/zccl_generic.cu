// Codec for streams whose tile size is not the 4096 elements the tuned kernels are built around (Section 3.5.2
// cuts the data into chunks of 5120 points; the tile size is a header field of the stream).  Plain kernels, one CTA
// per tile and one warp per block of 32, with the arithmetic of the tuned kernels' integer route: q = rint(x * r) by
// one fp32 multiplication and one conversion, deltas inside the tile, code length = bit length of the largest
// magnitude of a block, sign word and bit planes by ballots.  Compression takes three launches (tile sizes, their
// prefix with header and index, the blobs), decompression one.  Any tile size that is a multiple of 32 between
// 1024 and 8192 elements.
#include "zccl_internal.h"

namespace zccl {
namespace {

constexpr unsigned kFull = 0xFFFFFFFFu;
constexpr int kGenMaxBlocks = kGenericMaxTile / kBlock;   // 256

__device__ __forceinline__ uint32_t bitlen(uint32_t v) { return 32u - (uint32_t)__clz((int)v); }

// Delta of element e of a tile (its code minus its predecessor's; 0 for the first element and for the padding
// lanes of a ragged last block, which repeat the last element).  `t_abs` receives |x * r| for the range checks.
__device__ __forceinline__ int32_t delta_at(const float* __restrict__ xt, uint32_t e, uint32_t last, float r, float& t_abs,
                                            int32_t& q_out)
{
    const uint32_t ec = e < last ? e : last;
    const uint32_t em = e ? e - 1 : 0;
    const uint32_t ep = em < last ? em : last;
    const float t = __fmul_rn(__ldg(xt + ec), r), tp = __fmul_rn(__ldg(xt + ep), r);
    t_abs = fabsf(t);
    const int32_t q = __float2int_rn(t), qp = __float2int_rn(tp);
    q_out = q;
    return q - qp;
}

// Pass 1 (emit == 0): words of every tile's blob into sizes[].  Pass 3 (emit == 1): the blobs themselves, at the
// places the index (written by the scan in between) gives them.
__global__ void __launch_bounds__(256) generic_encode_kernel(const float* __restrict__ x, unsigned long long n, uint32_t T, uint32_t nT,
                                                             Params hp, int use_dev_params, uint32_t* __restrict__ sizes,
                                                             uint32_t* __restrict__ out, const uint32_t* __restrict__ go, int emit,
                                                             Workspace ws)
{
    __shared__ uint32_t Ls[kGenMaxBlocks];
    __shared__ uint32_t offs[kGenMaxBlocks + 1];
    __shared__ uint32_t wsum[8];
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const Params p = use_dev_params ? *ws.params : hp;
    if (!p.valid) return;
    if (emit && *go == 0) return;
    uint32_t status = 0;
    for (uint32_t t = blockIdx.x; t < nT; t += gridDim.x) {
        const unsigned long long start = (unsigned long long)t * T;
        const uint32_t len = (uint32_t)((n - start < (unsigned long long)T) ? (n - start) : (unsigned long long)T);
        const uint32_t nb = (len + kBlock - 1) / kBlock;
        const float* xt = x + start;
        float tmax = 0.0f;
        uint32_t words = 0;
        for (uint32_t b = warp; b < nb; b += 8) {
            float ta; int32_t q;
            const int32_t d = delta_at(xt, 32u * b + lane, len - 1, p.r, ta, q);
            tmax = fmaxf(tmax, ta);
            const uint32_t L = bitlen(__reduce_or_sync(kFull, (uint32_t)(d < 0 ? -d : d)));
            if (lane == 0) Ls[b] = L;
            words += L ? L + 1 : 0;
        }
#pragma unroll
        for (int s = 16; s; s >>= 1) tmax = fmaxf(tmax, __shfl_xor_sync(kFull, tmax, s));
        if (!(tmax < 1073741824.0f)) status |= kStRange;
        else if (tmax > 32768.5f) status |= kStPrecision;
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
                float ta; int32_t q0;
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
                float ta; int32_t q;
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
__global__ void __launch_bounds__(1024) generic_scan_kernel(const uint32_t* __restrict__ sizes, unsigned long long n, uint32_t T, uint32_t nT,
                                                            Params hp, int use_dev_params, uint32_t* __restrict__ out,
                                                            unsigned long long out_cap, size_t* __restrict__ out_bytes,
                                                            uint32_t* __restrict__ go, Workspace ws)
{
    __shared__ unsigned long long wtot[32];
    __shared__ unsigned long long carry_s;
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const Params p = use_dev_params ? *ws.params : hp;
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
        out[0] = kMagic; out[1] = kVersion;
        out[2] = (uint32_t)n; out[3] = (uint32_t)(n >> 32);
        out[4] = __float_as_uint(p.eb_abs); out[5] = __float_as_uint(p.s);
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
__global__ void __launch_bounds__(256) generic_decode_kernel(const uint32_t* __restrict__ in, unsigned long long cap_bytes, uint32_t T,
                                                             float* __restrict__ y, unsigned long long y_cap, Workspace ws)
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
    float s = 1.0f;
    if (ok) {
        n = (unsigned long long)__ldg(in + 2) | ((unsigned long long)__ldg(in + 3) << 32);
        s = __uint_as_float(__ldg(in + 5));
        nT = __ldg(in + 7);
        ok = __ldg(in + 0) == kMagic && __ldg(in + 1) == kVersion && __ldg(in + 6) == T && (n + T - 1) / T == nT &&
             cap_bytes >= (unsigned long long)kHeaderBytes + 4ull * nT && s > 0.0f && isfinite(s);
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
                y[start + e] = __fmul_rn(__int2float_rn(btot[e >> 5] + pre[e]), s);
        } else if (tid == 0) {
            atomicOr(ws.status, kStBadStream);
        }
        __syncthreads();
        if (tid == 0) bad_s = 0;
        __syncthreads();
    }
}

}  // namespace

cudaError_t launch_generic_encode(const float* x, unsigned long long n, uint32_t T, Params hp, bool device_params, uint32_t* sizes,
                                  uint32_t* go, uint32_t* out, unsigned long long out_cap, size_t* out_bytes, const Workspace& ws,
                                  int sm_count, cudaStream_t st)
{
    const uint32_t nT = (uint32_t)((n + T - 1) / T);
    const unsigned grid = nT < (unsigned)sm_count * 4u ? (nT ? nT : 1u) : (unsigned)sm_count * 4u;
    const int dp = device_params ? 1 : 0;
    count_launches(3);
    generic_encode_kernel<<<grid, 256, 0, st>>>(x, n, T, nT, hp, dp, sizes, out, go, 0, ws);
    generic_scan_kernel<<<1, 1024, 0, st>>>(sizes, n, T, nT, hp, dp, out, out_cap, out_bytes, go, ws);
    generic_encode_kernel<<<grid, 256, 0, st>>>(x, n, T, nT, hp, dp, sizes, out, go, 1, ws);
    return cudaGetLastError();
}

cudaError_t launch_generic_decode(const uint32_t* in, unsigned long long cap_bytes, uint32_t T, float* y, unsigned long long y_cap,
                                  const Workspace& ws, int sm_count, cudaStream_t st)
{
    const unsigned long long nT = (y_cap + T - 1) / T;
    const unsigned cap = (unsigned)sm_count * 4u;
    const unsigned grid = nT < cap ? (unsigned)(nT ? nT : 1) : cap;
    count_launches(1);
    generic_decode_kernel<<<grid, 256, 0, st>>>(in, cap_bytes, T, y, y_cap, ws);
    return cudaGetLastError();
}

}  // namespace zccl
