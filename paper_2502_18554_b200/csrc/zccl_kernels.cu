// fZ-light codec kernels for sm_100a: range reduction, bound resolution, encoder (plain and fused with a
// decode + add front end), decoder, and compressed-chunk copy.
//
// Work decomposition: one CTA of 256 threads handles one 4096-element tile at a time; each of its 8 warps owns
// 16 consecutive 32-element blocks, one element per lane, so a block's code length is a warp OR-reduction and
// each bit plane is one ballot.  Tiles are handed out by an atomic ticket, so a tile's predecessors in the
// placement scan (decoupled look-back over tile sizes) have always started before it.
#include "zccl_internal.h"

namespace zccl {

namespace {

constexpr unsigned kFull = 0xFFFFFFFFu;
constexpr int kSpinLimit = 1 << 20;   // polls of a predecessor's scan state before giving up (about a second)

__device__ __forceinline__ uint32_t f2key(float f)
{
    uint32_t u = __float_as_uint(f);
    return (u & 0x80000000u) ? ~u : (u | 0x80000000u);
}
__device__ __forceinline__ float key2f(uint32_t k)
{
    return __uint_as_float((k & 0x80000000u) ? (k & 0x7FFFFFFFu) : ~k);
}

__device__ __forceinline__ unsigned long long pack_state(uint32_t epoch, uint32_t inclusive, uint32_t words)
{
    return ((unsigned long long)epoch << 33) | ((unsigned long long)inclusive << 32) | words;
}

__device__ __forceinline__ unsigned long long ld_state(const unsigned long long* p)
{
    unsigned long long v;
    asm volatile("ld.relaxed.gpu.global.u64 %0, [%1];" : "=l"(v) : "l"(p) : "memory");
    return v;
}
__device__ __forceinline__ void st_state(unsigned long long* p, unsigned long long v)
{
    asm volatile("st.relaxed.gpu.global.u64 [%0], %1;" ::"l"(p), "l"(v) : "memory");
}

__device__ __forceinline__ uint32_t ldg_u32(const uint32_t* p) { return __ldg(p); }

// ------------------------------------------------------------------------------------------------ range (REL)

__global__ void __launch_bounds__(256) range_kernel(RangeBatch rb, Workspace ws)
{
    float lo = __int_as_float(0x7F800000), hi = __int_as_float(0xFF800000);
    const int j = blockIdx.y;
    const float* x = rb.x[j];
    const unsigned long long n = rb.n[j];
    const unsigned long long tid = (unsigned long long)blockIdx.x * blockDim.x + threadIdx.x;
    const unsigned long long nthreads = (unsigned long long)gridDim.x * blockDim.x;
    // peel to a 16-byte boundary, then 128-bit loads
    unsigned long long head = ((16u - (unsigned)((uintptr_t)x & 15u)) & 15u) >> 2;
    if (head > n) head = n;
    if (tid < head) { float v = x[tid]; lo = fminf(lo, v); hi = fmaxf(hi, v); }
    const unsigned long long nvec = (n - head) >> 2;
    const float4* xv = reinterpret_cast<const float4*>(x + head);
    for (unsigned long long i = tid; i < nvec; i += nthreads) {
        float4 v = __ldg(xv + i);
        lo = fminf(fminf(lo, v.x), fminf(v.y, fminf(v.z, v.w)));
        hi = fmaxf(fmaxf(hi, v.x), fmaxf(v.y, fmaxf(v.z, v.w)));
    }
    const unsigned long long tail0 = head + (nvec << 2);
    if (tail0 + tid < n) { float v = x[tail0 + tid]; lo = fminf(lo, v); hi = fmaxf(hi, v); }
#pragma unroll
    for (int d = 16; d; d >>= 1) {
        lo = fminf(lo, __shfl_xor_sync(kFull, lo, d));
        hi = fmaxf(hi, __shfl_xor_sync(kFull, hi, d));
    }
    __shared__ float s_lo[8], s_hi[8];
    if ((threadIdx.x & 31) == 0) { s_lo[threadIdx.x >> 5] = lo; s_hi[threadIdx.x >> 5] = hi; }
    __syncthreads();
    if (threadIdx.x == 0) {
        for (int w = 1; w < 8; ++w) { lo = fminf(lo, s_lo[w]); hi = fmaxf(hi, s_hi[w]); }
        if (n) {
            atomicMin(&ws.minmax[0], f2key(lo));
            atomicMax(&ws.minmax[1], f2key(hi));
        }
    }
}

// eb -> (eb_abs, s, r), the reading used throughout: eb_abs = eb * (max - min); step shrunk by 1 - 2^-6;
// r by one IEEE division.  Consumes and re-arms the min/max keys.
__global__ void resolve_kernel(int eb_mode, float eb, Workspace ws)
{
    if (threadIdx.x || blockIdx.x) return;
    Params p;
    p.valid = 1;
    float ea = eb;
    if (eb_mode == 1) {
        const uint32_t kmin = ws.minmax[0], kmax = ws.minmax[1];
        float range = 0.0f;
        if (kmin <= kmax) range = __fsub_rn(key2f(kmax), key2f(kmin));
        if (!(range > 0.0f) || !isfinite(range)) p.valid = 0;
        ea = __fmul_rn(eb, range);
        ws.minmax[0] = 0xFFFFFFFFu;
        ws.minmax[1] = 0u;
    }
    const float ebq = __fmul_rn(ea, 0.984375f);
    const float s = __fmul_rn(ebq, 2.0f);
    if (!(s > 0.0f) || !isfinite(s)) p.valid = 0;
    const float r = __fdiv_rn(1.0f, s);
    if (!isfinite(r)) p.valid = 0;
    p.eb_abs = ea; p.s = s; p.r = r;
    *ws.params = p;
    if (!p.valid) atomicOr(ws.status, kStDegenerate);
}

// ------------------------------------------------------------------------------------------------ stream header

struct StreamInfo {
    unsigned long long n;
    uint32_t nT;
    float eb_abs, s;
    bool ok;
};

__device__ __forceinline__ StreamInfo read_header(const uint32_t* in, unsigned long long cap_bytes)
{
    StreamInfo h;
    h.ok = false; h.n = 0; h.nT = 0; h.s = 1.0f; h.eb_abs = 0.0f;
    if (cap_bytes < (unsigned)kHeaderBytes) return h;
    const uint32_t magic = ldg_u32(in + 0), ver = ldg_u32(in + 1);
    const unsigned long long n = (unsigned long long)ldg_u32(in + 2) | ((unsigned long long)ldg_u32(in + 3) << 32);
    const float eb_abs = __uint_as_float(ldg_u32(in + 4)), s = __uint_as_float(ldg_u32(in + 5));
    const uint32_t T = ldg_u32(in + 6), nT = ldg_u32(in + 7);
    if (magic != kMagic || ver != kVersion || T != (uint32_t)kTile) return h;
    if ((n + kTile - 1) / kTile != nT) return h;
    if (cap_bytes < (unsigned long long)kHeaderBytes + 4ull * nT) return h;
    if (!(s > 0.0f) || !isfinite(s)) return h;
    h.n = n; h.nT = nT; h.eb_abs = eb_abs; h.s = s; h.ok = true;
    return h;
}

// ------------------------------------------------------------------------------------------------ tile decoder

// Decodes this warp's 16 blocks of tile `tile` into codes relative to the warp's first element:
// q[i] = sum of the deltas from the warp's first block up to this lane (the caller adds the outlier and the sums
// of the preceding warps).  Returns false, uniformly over the CTA, when the tile's blob is inconsistent.
__device__ __forceinline__ bool decode_tile_warp(const uint32_t* __restrict__ in, unsigned long long cap_bytes,
                                                 const StreamInfo& h, uint32_t tile, int warp, int lane,
                                                 int32_t (&q)[kBlocksPerWarp], int32_t& outlier)
{
    const uint32_t* idx = in + kHeaderWords;
    const uint32_t w_end = ldg_u32(idx + tile);
    const uint32_t w_beg = tile ? ldg_u32(idx + tile - 1) : 0u;
    const unsigned long long blob0 = (unsigned long long)kHeaderWords + h.nT;   // in words
    if (w_end < w_beg) return false;
    if ((blob0 + w_end) * 4ull > cap_bytes) return false;
    const unsigned long long start = (unsigned long long)tile * kTile;
    const uint32_t len = (uint32_t)((h.n - start < (unsigned long long)kTile) ? (h.n - start) : kTile);
    const uint32_t nb = (len + kBlock - 1) / kBlock;
    const uint32_t padw = (nb + 3) >> 2;
    const uint32_t words = w_end - w_beg;
    if (words < 1 + padw) return false;
    const uint32_t* blob = in + blob0 + w_beg;
    outlier = (int32_t)ldg_u32(blob);

    // code lengths: one word (4 blocks) per lane; sizes; warp-wide exclusive scan of the sizes
    uint32_t lw = ((uint32_t)lane < padw) ? ldg_u32(blob + 1 + lane) : 0u;
    const uint32_t L0 = lw & 0xFF, L1 = (lw >> 8) & 0xFF, L2 = (lw >> 16) & 0xFF, L3 = lw >> 24;
    bool bad = (L0 > 31) | (L1 > 31) | (L2 > 31) | (L3 > 31);
    // blocks at or beyond nb must have zero code length (they are padding of the code-length area)
    const uint32_t b0 = 4u * lane;
    if ((b0 + 0 >= nb && L0) || (b0 + 1 >= nb && L1) || (b0 + 2 >= nb && L2) || (b0 + 3 >= nb && L3)) bad = true;
    const uint32_t z0 = L0 ? L0 + 1 : 0, z1 = L1 ? L1 + 1 : 0, z2 = L2 ? L2 + 1 : 0, z3 = L3 ? L3 + 1 : 0;
    const uint32_t lane_sum = z0 + z1 + z2 + z3;
    uint32_t incl = lane_sum;
#pragma unroll
    for (int d = 1; d < 32; d <<= 1) {
        uint32_t t = __shfl_up_sync(kFull, incl, d);
        if (lane >= d) incl += t;
    }
    const uint32_t total = __shfl_sync(kFull, incl, 31);
    bad = __any_sync(kFull, bad);
    if (bad || 1 + padw + total != words) return false;
    const uint32_t o0 = incl - lane_sum, o1 = o0 + z0, o2 = o1 + z1, o3 = o2 + z2;
    const uint32_t* payload = blob + 1 + padw;

    // fetch: lane k of a block reads word k of the block's payload (sign word, then planes)
    uint32_t word[kBlocksPerWarp];
    uint32_t Ls[kBlocksPerWarp];
#pragma unroll
    for (int i = 0; i < kBlocksPerWarp; ++i) {
        const int src = 4 * warp + (i >> 2);
        const uint32_t lwi = __shfl_sync(kFull, lw, src);
        const uint32_t L = (lwi >> (8 * (i & 3))) & 0xFF;
        const uint32_t osel = (i & 3) == 0 ? o0 : (i & 3) == 1 ? o1 : (i & 3) == 2 ? o2 : o3;
        const uint32_t off = __shfl_sync(kFull, osel, src);
        Ls[i] = L;
        word[i] = (L && (uint32_t)lane <= L) ? ldg_u32(payload + off + lane) : 0u;
    }
    int32_t carry = 0;
#pragma unroll
    for (int i = 0; i < kBlocksPerWarp; ++i) {
        const uint32_t L = Ls[i];
        int32_t v = 0;
        if (L) {   // uniform over the warp
            const uint32_t sign = __shfl_sync(kFull, word[i], 0);
            uint32_t mag = 0;
            for (uint32_t k = 0; k < L; ++k) {
                const uint32_t plane = __shfl_sync(kFull, word[i], k + 1);
                mag |= ((plane >> lane) & 1u) << k;
            }
            v = ((sign >> lane) & 1u) ? -(int32_t)mag : (int32_t)mag;
#pragma unroll
            for (int d = 1; d < 32; d <<= 1) {
                int32_t t = __shfl_up_sync(kFull, v, d);
                if (lane >= d) v += t;
            }
        }
        q[i] = carry + v;
        carry = __shfl_sync(kFull, q[i], 31);
    }
    return true;
}

// ------------------------------------------------------------------------------------------------ encoder

struct EncodeShared {
    uint32_t stage[1 + kBlocksPerTile / 4 + kBlocksPerTile * kBlock];   // a tile's blob, worst case
    uint32_t warp_words[kWarps];
    int32_t warp_lastq[kWarps];
    int32_t warp_sum[2][kWarps];
    uint32_t ticket;
    uint32_t excl;
    uint32_t skip;
};

template <int MODE>
__global__ void __launch_bounds__(kThreads, 3) encode_kernel(JobBatch jb, Workspace ws, Params hp, int use_dev_params)
{
    __shared__ EncodeShared sh;
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const uint32_t epoch = *reinterpret_cast<volatile uint32_t*>(ws.epoch);
    uint32_t status = 0;

    Params prm = hp;
    if (MODE == kEncodeRaw && use_dev_params) prm = *ws.params;

    for (;;) {
        __syncthreads();
        if (tid == 0) sh.ticket = atomicAdd(ws.ticket, 1u);
        __syncthreads();
        const uint32_t ticket = sh.ticket;
        if (ticket >= jb.total_tiles) break;
        int j = 0;
#pragma unroll 1
        for (int k = 1; k < jb.count; ++k) if (jb.job[k].tile_begin <= ticket) j = k;
        const Job& job = jb.job[j];
        const uint32_t tile = ticket - job.tile_begin;
        const unsigned long long n = job.n;
        const uint32_t nT = (uint32_t)((n + kTile - 1) / kTile);
        unsigned long long* my_state = ws.tile_state + ticket;

        bool tile_ok = true;
        float s = prm.s, r = prm.r, eb_abs = prm.eb_abs;
        StreamInfo h1, h2;
        if (MODE == kEncodeFused) {
            h1 = read_header(job.in_c, job.in_cap);
            tile_ok = h1.ok && h1.n == n;
            if (job.in_c2) {
                h2 = read_header(job.in_c2, job.in2_cap);
                tile_ok = tile_ok && h2.ok && h2.n == n && __float_as_uint(h2.s) == __float_as_uint(h1.s);
            }
            s = h1.s; eb_abs = h1.eb_abs;
            r = __fdiv_rn(1.0f, s);
            if (!tile_ok) status |= kStBadStream;
        } else {
            tile_ok = prm.valid != 0;
        }

        // a job with no elements still owns one ticket: it writes the header and the length
        if (n == 0 || !tile_ok) {
            if (tid == 0) {
                st_state(my_state, pack_state(epoch, 1u, 0u));
                if (tile == 0) {
                    if (tile_ok && job.out_cap >= (unsigned)kHeaderBytes) {
                        uint32_t* o = job.out;
                        o[0] = kMagic; o[1] = kVersion; o[2] = 0; o[3] = 0;
                        o[4] = __float_as_uint(eb_abs); o[5] = __float_as_uint(s); o[6] = kTile; o[7] = 0;
                        *job.out_bytes = kHeaderBytes;
                    } else {
                        *job.out_bytes = 0;
                    }
                }
            }
            continue;
        }

        const unsigned long long start = (unsigned long long)tile * kTile;
        const uint32_t len = (uint32_t)((n - start < (unsigned long long)kTile) ? (n - start) : kTile);
        const uint32_t nb = (len + kBlock - 1) / kBlock;
        const uint32_t padw = (nb + 3) >> 2;
        const unsigned long long last = n - 1;

        // ---- values of this warp's 16 blocks, one element per lane; lanes past the end repeat the last element
        float v[kBlocksPerWarp];
        const unsigned long long e0 = start + (unsigned)(warp * kBlocksPerWarp * kBlock + lane);
        if (MODE == kEncodeRaw) {
            const float* __restrict__ x = job.x;
#pragma unroll
            for (int i = 0; i < kBlocksPerWarp; ++i) {
                unsigned long long e = e0 + (unsigned)(i * kBlock);
                v[i] = __ldg(x + (e < last ? e : last));
            }
        } else {
            int32_t qa[kBlocksPerWarp], oa = 0;
            bool ok = decode_tile_warp(job.in_c, job.in_cap, h1, tile, warp, lane, qa, oa);
            int32_t qb[kBlocksPerWarp], ob = 0;
            if (job.in_c2) ok = decode_tile_warp(job.in_c2, job.in2_cap, h2, tile, warp, lane, qb, ob) && ok;
            if (lane == 31) {
                sh.warp_sum[0][warp] = qa[kBlocksPerWarp - 1];
                if (job.in_c2) sh.warp_sum[1][warp] = qb[kBlocksPerWarp - 1];
            }
            __syncthreads();
            if (!ok) {   // uniform over the CTA
                status |= kStBadStream;
                // keep the scan consistent for the tiles that follow: publish an empty tile, write nothing
                if (tid == 0) st_state(my_state, pack_state(epoch, tile == 0 ? 1u : 0u, 0u));
                if (tid == 0 && tile == nT - 1) *job.out_bytes = 0;
                continue;
            }
            int32_t base_a = oa, base_b = ob;
            for (int w = 0; w < warp; ++w) { base_a += sh.warp_sum[0][w]; if (job.in_c2) base_b += sh.warp_sum[1][w]; }
            const float* __restrict__ loc = job.x;
#pragma unroll
            for (int i = 0; i < kBlocksPerWarp; ++i) {
                unsigned long long e = e0 + (unsigned)(i * kBlock);
                if (e > last) e = last;
                const float xa = __fmul_rn(__int2float_rn(base_a + qa[i]), s);
                float xb;
                if (job.in_c2) xb = __fmul_rn(__int2float_rn(base_b + qb[i]), s);
                else xb = __ldg(loc + e);
                v[i] = __fadd_rn(xa, xb);
            }
        }

        // ---- quantise (the multiplication), keep the largest |x * r| for the range / precision checks
        int32_t q[kBlocksPerWarp];
        float tmax = 0.0f;
#pragma unroll
        for (int i = 0; i < kBlocksPerWarp; ++i) {
            const float t = __fmul_rn(v[i], r);
            tmax = fmaxf(tmax, fabsf(t));
            q[i] = __float2int_rn(t);
        }
        if (!(tmax < 1073741824.0f)) status |= kStRange;
        else if (tmax > 32768.5f) status |= kStPrecision;

        if (MODE == kEncodeFused && job.y != nullptr) {   // uncompressed copy of the sum for the chunk's owner
            float* __restrict__ y = job.y;
            const bool deq = (job.flags & 1u) != 0;
#pragma unroll
            for (int i = 0; i < kBlocksPerWarp; ++i) {
                unsigned long long e = e0 + (unsigned)(i * kBlock);
                if (e <= last) y[e] = deq ? __fmul_rn(__int2float_rn(q[i]), s) : v[i];
            }
        }

        if (lane == 31) sh.warp_lastq[warp] = q[kBlocksPerWarp - 1];
        __syncthreads();

        // ---- 1-D Lorenzo deltas, code lengths
        uint32_t mag[kBlocksPerWarp];
        uint32_t sgn[kBlocksPerWarp];
        uint32_t Ls[kBlocksPerWarp];
        int32_t prev_last = (warp == 0) ? __shfl_sync(kFull, q[0], 0) : sh.warp_lastq[warp - 1];
#pragma unroll
        for (int i = 0; i < kBlocksPerWarp; ++i) {
            const int32_t src = (lane == 31) ? prev_last : q[i];
            const int32_t prev = __shfl_sync(kFull, src, (lane + 31) & 31);
            const int32_t d = q[i] - prev;
            prev_last = q[i];     // only lane 31's copy is consumed by the next block
            const uint32_t a = (uint32_t)(d < 0 ? -d : d);
            const uint32_t m = __reduce_or_sync(kFull, a);
            uint32_t L = 32u - (uint32_t)__clz((int)m);
            L = L > 31u ? 31u : L;
            mag[i] = a;
            sgn[i] = __ballot_sync(kFull, d < 0);
            Ls[i] = L;
        }

        // ---- sizes: serial exclusive scan over this warp's 16 blocks (uniform), then across warps
        uint32_t off[kBlocksPerWarp];
        uint32_t wsum = 0;
#pragma unroll
        for (int i = 0; i < kBlocksPerWarp; ++i) { off[i] = wsum; wsum += Ls[i] ? Ls[i] + 1 : 0; }
        if (lane == 0) sh.warp_words[warp] = wsum;
        // code-length bytes of this warp's blocks: 4 words of the code-length area
        if (lane < 4) {
            uint32_t wv = 0;
#pragma unroll
            for (int i = 0; i < kBlocksPerWarp; ++i)
                if ((i >> 2) == lane) wv |= Ls[i] << (8 * (i & 3));
            const uint32_t widx = 4 * warp + lane;
            if (widx < padw) sh.stage[1 + widx] = wv;
        }
        if (tid == 0) sh.stage[0] = (uint32_t)q[0];   // the outlier
        __syncthreads();
        uint32_t wbase = 1 + padw, total = 1 + padw;
#pragma unroll
        for (int w = 0; w < kWarps; ++w) {
            const uint32_t ww = sh.warp_words[w];
            if (w < warp) wbase += ww;
            total += ww;
        }
        if (tid == 0) st_state(my_state, pack_state(epoch, tile == 0 ? 1u : 0u, total));

        // ---- fixed-length encoding: sign word and one ballot per bit plane into the staged blob
#pragma unroll
        for (int i = 0; i < kBlocksPerWarp; ++i) {
            const uint32_t L = Ls[i];
            if (L) {   // uniform over the warp
                uint32_t* dst = sh.stage + wbase + off[i];
                uint32_t mine = sgn[i];
                for (uint32_t k = 0; k < L; ++k) {
                    const uint32_t plane = __ballot_sync(kFull, (mag[i] >> k) & 1u);
                    if ((uint32_t)lane == k + 1) mine = plane;
                }
                if ((uint32_t)lane <= L) dst[lane] = mine;
            }
        }

        // ---- placement: decoupled look-back over the preceding tiles of this job (warp 0)
        if (warp == 0) {
            uint32_t excl = 0, skip = 0;
            if (tile != 0) {
                long long pos = (long long)ticket - 1;
                const long long lo = (long long)job.tile_begin;
                int budget = kSpinLimit;
                for (;;) {
                    const long long at = pos - lane;
                    unsigned long long st = pack_state(epoch, 1u, 0u);   // before the job's first tile: prefix 0
                    if (at >= lo) st = ld_state(ws.tile_state + at);
                    const bool valid = (uint32_t)(st >> 33) == epoch;
                    const uint32_t vmask = __ballot_sync(kFull, valid);
                    const uint32_t imask = __ballot_sync(kFull, valid && ((st >> 32) & 1ull));
                    const int first = imask ? (__ffs((int)imask) - 1) : 31;
                    const uint32_t need = (first == 31) ? kFull : ((2u << first) - 1u);
                    if ((vmask & need) != need) {
                        if (--budget == 0) { skip = 1; status |= kStTimeout; break; }
                        __nanosleep(64);
                        continue;
                    }
                    const uint32_t contrib = (lane <= first) ? (uint32_t)st : 0u;
                    excl += __reduce_add_sync(kFull, contrib);
                    if (imask) break;
                    pos -= 32;
                }
                if (lane == 0) st_state(my_state, pack_state(epoch, 1u, excl + total));
            }
            if (lane == 0) { sh.excl = excl; sh.skip = skip; }
        }
        __syncthreads();

        // ---- copy the staged blob to its place; index entry; header and length
        const uint32_t excl = sh.excl;
        const unsigned long long blob_word0 = (unsigned long long)kHeaderWords + nT + excl;
        const bool fits = (blob_word0 + total) * 4ull <= job.out_cap;
        if (!fits) status |= kStCapacity;
        if (fits && !sh.skip) {
            uint32_t* __restrict__ o = job.out + blob_word0;
            for (uint32_t i = tid; i < total; i += kThreads) o[i] = sh.stage[i];
            if (tid == 0) job.out[kHeaderWords + tile] = excl + total;
        }
        if (tile == 0 && tid < kHeaderWords) {
            uint32_t hv;
            switch (tid) {
                case 0: hv = kMagic; break;
                case 1: hv = kVersion; break;
                case 2: hv = (uint32_t)n; break;
                case 3: hv = (uint32_t)(n >> 32); break;
                case 4: hv = __float_as_uint(eb_abs); break;
                case 5: hv = __float_as_uint(s); break;
                case 6: hv = kTile; break;
                default: hv = nT; break;
            }
            job.out[tid] = hv;
        }
        if (tile == nT - 1 && tid == 0) *job.out_bytes = (size_t)((blob_word0 + total) * 4ull);
    }

    if (status) atomicOr(ws.status, status);
    __syncthreads();
    if (tid == 0) {
        __threadfence();
        const uint32_t prev = atomicAdd(ws.done, 1u);
        if (prev == gridDim.x - 1) {   // every CTA has drawn its last ticket: re-arm for the next launch
            *ws.ticket = 0;
            *ws.done = 0;
            uint32_t e = (epoch + 1u) & 0x7FFFFFFFu;
            *ws.epoch = e ? e : 1u;
        }
    }
}

// ------------------------------------------------------------------------------------------------ decoder

__global__ void __launch_bounds__(kThreads, 3) decode_kernel(JobBatch jb, Workspace ws)
{
    __shared__ int32_t s_warp_sum[kWarps];
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    uint32_t status = 0;
    for (uint32_t g = blockIdx.x; g < jb.total_tiles; g += gridDim.x) {
        int j = 0;
#pragma unroll 1
        for (int k = 1; k < jb.count; ++k) if (jb.job[k].tile_begin <= g) j = k;
        const Job& job = jb.job[j];
        const uint32_t tile = g - job.tile_begin;
        const StreamInfo h = read_header(job.in_c, job.in_cap);
        if (!h.ok) { status |= kStBadStream; continue; }
        if (h.n > job.n) { status |= kStCapacity; continue; }
        if (tile >= h.nT) continue;
        int32_t q[kBlocksPerWarp], outlier = 0;
        const bool ok = decode_tile_warp(job.in_c, job.in_cap, h, tile, warp, lane, q, outlier);
        __syncthreads();   // previous iteration's readers of s_warp_sum are done
        if (lane == 31) s_warp_sum[warp] = q[kBlocksPerWarp - 1];
        __syncthreads();
        if (!ok) { status |= kStBadStream; continue; }
        int32_t base = outlier;
        for (int w = 0; w < warp; ++w) base += s_warp_sum[w];
        const unsigned long long e0 = (unsigned long long)tile * kTile + (unsigned)(warp * kBlocksPerWarp * kBlock + lane);
        float* __restrict__ y = job.y;
#pragma unroll
        for (int i = 0; i < kBlocksPerWarp; ++i) {
            const unsigned long long e = e0 + (unsigned)(i * kBlock);
            if (e < h.n) y[e] = __fmul_rn(__int2float_rn(base + q[i]), h.s);
        }
    }
    if (status) atomicOr(ws.status, status);
}

// ------------------------------------------------------------------------------------------------ blob copy

// One forwarding hop of compressed bytes whose length lives on the device (grid.y = job).
__global__ void __launch_bounds__(256) copy_kernel(CopyBatch cb, Workspace ws)
{
    const CopyJob& job = cb.job[blockIdx.y];
    const unsigned long long bytes = *job.bytes;
    if (bytes > job.cap) {
        if (threadIdx.x == 0 && blockIdx.x == 0) { atomicOr(ws.status, kStCapacity); if (job.bytes_out) *job.bytes_out = 0; }
        return;
    }
    const unsigned long long words = bytes >> 2;
    const unsigned long long tid = (unsigned long long)blockIdx.x * blockDim.x + threadIdx.x;
    const unsigned long long nth = (unsigned long long)gridDim.x * blockDim.x;
    const bool aligned = ((((uintptr_t)job.src) | ((uintptr_t)job.dst)) & 15u) == 0;
    unsigned long long done_words = 0;
    if (aligned) {
        const unsigned long long nv = words >> 2;
        const uint4* s4 = reinterpret_cast<const uint4*>(job.src);
        uint4* d4 = reinterpret_cast<uint4*>(job.dst);
        for (unsigned long long i = tid; i < nv; i += nth) d4[i] = __ldg(s4 + i);
        done_words = nv << 2;
    }
    for (unsigned long long i = done_words + tid; i < words; i += nth) job.dst[i] = __ldg(job.src + i);
    if (tid == 0 && job.bytes_out) *job.bytes_out = (size_t)bytes;
}

int g_encode_ctas_per_sm = 0, g_decode_ctas_per_sm = 0;
unsigned long long g_launches = 0;   // kernels launched by this library in this process

}  // namespace

// ------------------------------------------------------------------------------------------------ launchers

unsigned long long launch_count() { return g_launches; }

cudaError_t launch_range(const RangeBatch& rb, const Workspace& ws, int sm_count, cudaStream_t st)
{
    if (rb.count <= 0) return cudaSuccess;
    unsigned long long nmax = 0;
    for (int j = 0; j < rb.count; ++j) nmax = rb.n[j] > nmax ? rb.n[j] : nmax;
    unsigned long long want = (nmax / 4 + 255) / 256;
    unsigned per = (unsigned)((sm_count * 8 + rb.count - 1) / rb.count);
    unsigned gx = (unsigned)(want < per ? (want ? want : 1) : per);
    ++g_launches;
    range_kernel<<<dim3(gx, rb.count), 256, 0, st>>>(rb, ws);
    return cudaGetLastError();
}

cudaError_t launch_resolve(int eb_mode, float eb, const Workspace& ws, cudaStream_t st)
{
    ++g_launches;
    resolve_kernel<<<1, 32, 0, st>>>(eb_mode, eb, ws);
    return cudaGetLastError();
}

cudaError_t launch_encode(const JobBatch& jb, EncodeMode mode, const Workspace& ws, bool device_params,
                          Params host_params, int sm_count, cudaStream_t st)
{
    if (jb.total_tiles == 0) return cudaSuccess;
    if (g_encode_ctas_per_sm == 0) {
        int a = 0, b = 0;
        cudaOccupancyMaxActiveBlocksPerMultiprocessor(&a, encode_kernel<kEncodeRaw>, kThreads, 0);
        cudaOccupancyMaxActiveBlocksPerMultiprocessor(&b, encode_kernel<kEncodeFused>, kThreads, 0);
        g_encode_ctas_per_sm = (a < b ? a : b) > 0 ? (a < b ? a : b) : 1;
    }
    unsigned long long cap = (unsigned long long)sm_count * g_encode_ctas_per_sm;
    unsigned grid = (unsigned)(jb.total_tiles < cap ? jb.total_tiles : cap);
    ++g_launches;
    if (mode == kEncodeRaw)
        encode_kernel<kEncodeRaw><<<grid, kThreads, 0, st>>>(jb, ws, host_params, device_params ? 1 : 0);
    else
        encode_kernel<kEncodeFused><<<grid, kThreads, 0, st>>>(jb, ws, host_params, 0);
    return cudaGetLastError();
}

cudaError_t launch_decode(const JobBatch& jb, const Workspace& ws, int sm_count, cudaStream_t st)
{
    if (jb.total_tiles == 0) return cudaSuccess;
    if (g_decode_ctas_per_sm == 0) {
        int a = 0;
        cudaOccupancyMaxActiveBlocksPerMultiprocessor(&a, decode_kernel, kThreads, 0);
        g_decode_ctas_per_sm = a > 0 ? a : 1;
    }
    unsigned long long cap = (unsigned long long)sm_count * g_decode_ctas_per_sm;
    unsigned grid = (unsigned)(jb.total_tiles < cap ? jb.total_tiles : cap);
    ++g_launches;
    decode_kernel<<<grid, kThreads, 0, st>>>(jb, ws);
    return cudaGetLastError();
}

cudaError_t launch_copy(const CopyBatch& cb, const Workspace& ws, int sm_count, cudaStream_t st)
{
    if (cb.count <= 0) return cudaSuccess;
    unsigned gx = (unsigned)((sm_count * 4 + cb.count - 1) / cb.count);
    ++g_launches;
    copy_kernel<<<dim3(gx ? gx : 1, cb.count), 256, 0, st>>>(cb, ws);
    return cudaGetLastError();
}

}  // namespace zccl
