// Auxiliary kernels of the fZ-light path for sm_100a: value range and bound resolution, compressed-chunk copies,
// the division of the Average, stream statistics and quality metrics, with their launchers.  The codec itself
// (encoder, decoder, fused hop) lives in zccl_codec.cu.
#include "zccl_device.cuh"

#include <atomic>

namespace zccl {

namespace {


// ------------------------------------------------------------------------------------------------ range (REL)

// eb -> (eb_abs, s, r), the reading used throughout: eb_abs = eb * (max - min); step shrunk by 1 - 2^-6;
// r by one IEEE division.  Consumes and re-arms the min/max keys.  One thread.
__device__ void resolve_from_range(float eb, float range, const Workspace& ws, float* eb_abs_out)
{
    Params p;
    p.valid = 1;
    if (!(range > 0.0f) || !isfinite(range)) p.valid = 0;
    const float ea = __fmul_rn(eb, range);
    const float ebq = __fmul_rn(ea, 0.984375f);
    const float s = __fmul_rn(ebq, 2.0f);
    if (!(s > 0.0f) || !isfinite(s)) p.valid = 0;
    const float r = __fdiv_rn(1.0f, s);
    if (!isfinite(r)) p.valid = 0;
    p.eb_abs = ea; p.s = s; p.r = r;
    *ws.params = p;
    if (eb_abs_out) *eb_abs_out = p.valid ? ea : 0.0f;
    if (!p.valid) atomicOr(ws.status, kStDegenerate);
}
__device__ void resolve_params(float eb, const Workspace& ws)
{
    const uint32_t kmin = *reinterpret_cast<volatile uint32_t*>(ws.minmax + 0);
    const uint32_t kmax = *reinterpret_cast<volatile uint32_t*>(ws.minmax + 1);
    float range = 0.0f;
    if (kmin <= kmax) range = __fsub_rn(key2f(kmax), key2f(kmin));
    ws.minmax[0] = 0xFFFFFFFFu;
    ws.minmax[1] = 0u;
    resolve_from_range(eb, range, ws, nullptr);
}

// The same from a (min, max) pair the caller has on the device: a rank's own pair combined with its peers'.
__global__ void resolve_range_kernel(const float* __restrict__ minmax, float eb, Workspace ws, float* eb_abs_out)
{
    pdl_enter();
    if (threadIdx.x == 0 && blockIdx.x == 0) {
        const float lo = minmax[0], hi = minmax[1];
        resolve_from_range(eb, lo <= hi ? __fsub_rn(hi, lo) : 0.0f, ws, eb_abs_out);
    }
}

// Hands the minimum and maximum to the caller (out[0] = min, out[1] = max; +inf, -inf when nothing was scanned)
// and re-arms the keys.  A rank of a real ring combines these with its peers' before it resolves the bound
// (Section 3.2: one bound per collective).  One thread.
__device__ void export_range(const Workspace& ws, float* out)
{
    const uint32_t kmin = *reinterpret_cast<volatile uint32_t*>(ws.minmax + 0);
    const uint32_t kmax = *reinterpret_cast<volatile uint32_t*>(ws.minmax + 1);
    const bool any = kmin <= kmax;
    out[0] = any ? key2f(kmin) : __int_as_float(0x7F800000);
    out[1] = any ? key2f(kmax) : __int_as_float(0xFF800000);
    ws.minmax[0] = 0xFFFFFFFFu;
    ws.minmax[1] = 0u;
}

// Minimum and maximum of up to kMaxJobs arrays into the workspace's two ordered keys.  With rb.finish set, the
// last CTA of the launch to get there turns the keys into the bound (kRangeResolve) or hands them out
// (kRangeExport), so that a relative bound costs one launch in front of the encoder.
__global__ void __launch_bounds__(256) range_kernel(RangeBatch rb, Workspace ws)
{
    pdl_enter();
    float lo = __int_as_float(0x7F800000), hi = __int_as_float(0xFF800000);
    const int j = blockIdx.y;
    const float* x = rb.x[j];
    const unsigned long long n = rb.n[j];
    const unsigned long long tid = (unsigned long long)blockIdx.x * blockDim.x + threadIdx.x;
    const unsigned long long nthreads = (unsigned long long)gridDim.x * blockDim.x;
    // peel to a 16-byte boundary, then 128-bit loads, four of them in flight per thread
    unsigned long long head = ((16u - (unsigned)((uintptr_t)x & 15u)) & 15u) >> 2;
    if (head > n) head = n;
    if (tid < head) { float v = x[tid]; lo = fminf(lo, v); hi = fmaxf(hi, v); }
    const unsigned long long nvec = (n - head) >> 2;
    const float4* xv = reinterpret_cast<const float4*>(x + head);
    unsigned long long i = tid;
    for (; i + 3 * nthreads < nvec; i += 4 * nthreads) {
        const float4 a = __ldg(xv + i), b = __ldg(xv + i + nthreads), c = __ldg(xv + i + 2 * nthreads),
                     d = __ldg(xv + i + 3 * nthreads);
        lo = fminf(fminf(fminf(lo, a.x), fminf(a.y, fminf(a.z, a.w))), fminf(fminf(b.x, b.y), fminf(b.z, b.w)));
        hi = fmaxf(fmaxf(fmaxf(hi, a.x), fmaxf(a.y, fmaxf(a.z, a.w))), fmaxf(fmaxf(b.x, b.y), fmaxf(b.z, b.w)));
        lo = fminf(fminf(fminf(lo, c.x), fminf(c.y, fminf(c.z, c.w))), fminf(fminf(d.x, d.y), fminf(d.z, d.w)));
        hi = fmaxf(fmaxf(fmaxf(hi, c.x), fmaxf(c.y, fmaxf(c.z, c.w))), fmaxf(fmaxf(d.x, d.y), fmaxf(d.z, d.w)));
    }
    for (; i < nvec; i += nthreads) {
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
        if (rb.finish != kRangeOnly) {
            __threadfence();
            if (atomicAdd(ws.done, 1u) == gridDim.x * gridDim.y - 1u) {   // every CTA's keys are in
                __threadfence();
                *ws.done = 0;
                if (rb.finish == kRangeResolve) resolve_params(rb.eb, ws);
                else export_range(ws, rb.out);
            }
        }
    }
}


// ------------------------------------------------------------------------------------------------ blob copy

// One forwarding hop of compressed bytes whose length lives on the device (grid.y = job).
__device__ __forceinline__ void copy_job(const CopyJob& job, const Workspace& ws)
{
    const unsigned long long bytes = job.bytes ? *job.bytes : job.fixed_bytes;
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
__global__ void __launch_bounds__(256) copy_kernel(CopyBatch cb, Workspace ws)
{
    pdl_enter();
    copy_job(cb.job[blockIdx.y], ws);
}

// Every forwarding hop of an Allgather stage (grid.y = chain).  A thread carries its 16-byte pieces through all the
// hops: each hop loads the piece from where the previous hop stored it (the same thread's own store, so no
// synchronisation is needed) and stores it into the next rank's slot.
// Rows of the grid beyond the chains are plain copies (`extra`): what else a collective has to move at that point goes
// along in the same launch.
__global__ void __launch_bounds__(256) copy_chain_kernel(ChainBatch cb, CopyBatch extra, Workspace ws)
{
    pdl_enter();
    if ((int)blockIdx.y >= cb.count) {
        copy_job(extra.job[blockIdx.y - cb.count], ws);
        return;
    }
    const ChainJob& job = cb.job[blockIdx.y];
    const unsigned long long bytes = *job.bytes;
    const unsigned long long tid = (unsigned long long)blockIdx.x * blockDim.x + threadIdx.x;
    const unsigned long long nth = (unsigned long long)gridDim.x * blockDim.x;
    const bool fits = bytes <= cb.slot_bytes;
    const bool ring = cb.hops >= 0;
    const int hops = ring ? cb.hops : job.hops;
    auto rank_of = [&](int h) { return ring ? (job.first_rank + h) % cb.N : (int)((job.path >> (8 * h)) & 0xFFu); };
    if (tid == 0) {
        if (!fits) atomicOr(ws.status, kStCapacity);
        for (int h = 0; h < hops; ++h)
            cb.sizes[(size_t)rank_of(h) * cb.N + job.chunk] = fits ? (size_t)bytes : 0;
    }
    if (!fits) return;
    const unsigned long long words = bytes >> 2;
    const unsigned long long nv = ((((uintptr_t)job.src0) & 15u) == 0) ? (words >> 2) : 0;   // slots are 256-byte aligned
    for (unsigned long long i = tid; i < nv; i += nth) {
        uint4 v = __ldg(reinterpret_cast<const uint4*>(job.src0) + i);
        for (int h = 0; h < hops; ++h) {
            uint4* d = reinterpret_cast<uint4*>(cb.slots + ((size_t)rank_of(h) * cb.N + job.chunk) * cb.slot_bytes) + i;
            *d = v;
            if (h + 1 < hops) asm volatile("ld.global.v4.u32 {%0, %1, %2, %3}, [%4];" : "=r"(v.x), "=r"(v.y), "=r"(v.z), "=r"(v.w) : "l"(d) : "memory");
        }
    }
    for (unsigned long long i = (nv << 2) + tid; i < words; i += nth) {
        uint32_t v = __ldg(job.src0 + i);
        for (int h = 0; h < hops; ++h) {
            uint32_t* d = reinterpret_cast<uint32_t*>(cb.slots + ((size_t)rank_of(h) * cb.N + job.chunk) * cb.slot_bytes) + i;
            *d = v;
            if (h + 1 < hops) asm volatile("ld.global.u32 %0, [%1];" : "=r"(v) : "l"(d) : "memory");
        }
    }
}

// y = y / divisor, element by element (Average = Sum / N at the end of the Allreduce).
__global__ void __launch_bounds__(256) scale_kernel(ScaleBatch sb)
{
    pdl_enter();
    float* __restrict__ y = sb.y[blockIdx.y];
    const unsigned long long tid = (unsigned long long)blockIdx.x * blockDim.x + threadIdx.x;
    const unsigned long long nth = (unsigned long long)gridDim.x * blockDim.x;
    for (unsigned long long i = tid; i < sb.n; i += nth) y[i] = __fdiv_rn(y[i], sb.divisor);
}

// ------------------------------------------------------------------------------------------------ stream statistics

// Histogram of the code lengths of a stream (hist[L], L = 0..31: blocks stored with code length L; hist[32]: blocks),
// from which the share of constant blocks (L = 0) and the mean code length follow.  One warp per tile: it finds the
// tile's blob through the index, reads the code-length bytes behind the outlier (a word of four per lane) and
// counts them in shared memory; every CTA adds its counts to the result at the end.
__global__ void __launch_bounds__(256) stream_stats_kernel(const uint32_t* __restrict__ in, unsigned long long cap_bytes,
                                                           unsigned long long* __restrict__ hist, Workspace ws)
{
    pdl_enter();
    __shared__ unsigned int cnt[33];
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    if (tid < 33) cnt[tid] = 0;
    __syncthreads();
    const StreamInfo h = read_header(in, cap_bytes);
    bool bad = !h.ok;
    if (h.ok) {
        const unsigned long long blob0 = (unsigned long long)kHeaderWords + h.nT;
        const uint32_t total_w = h.nT ? ldg_u32(in + kHeaderWords + h.nT - 1) : 0;
        if ((blob0 + total_w) * 4ull > cap_bytes) bad = true;
        const unsigned long long warps = (unsigned long long)gridDim.x * kWarps;
        for (unsigned long long t = (unsigned long long)blockIdx.x * kWarps + warp; !bad && t < h.nT; t += warps) {
            const uint32_t w_beg = t ? ldg_u32(in + kHeaderWords + t - 1) : 0, w_end = ldg_u32(in + kHeaderWords + t);
            const unsigned long long left = h.n - t * kTile;
            const uint32_t nb = (uint32_t)(((left < (unsigned long long)kTile ? left : (unsigned long long)kTile) + kBlock - 1) / kBlock);
            const uint32_t lw = (nb + 3) >> 2;                         // words of code-length bytes
            if (w_end < w_beg || w_end > total_w || w_end - w_beg < 1 + lw) { bad = true; break; }
            if ((uint32_t)lane < lw) {
                const uint32_t word = ldg_u32(in + blob0 + w_beg + 1 + lane);
#pragma unroll
                for (int k = 0; k < 4; ++k) {
                    if (4u * lane + k < nb) {
                        const uint32_t L = (word >> (8 * k)) & 0xFFu;
                        if (L > 31u) bad = true;
                        else { atomicAdd(&cnt[L], 1u); atomicAdd(&cnt[32], 1u); }
                    }
                }
            }
        }
    }
    if (__any_sync(kFull, bad) && lane == 0) atomicOr(ws.status, kStBadStream);
    __syncthreads();
    if (tid < 33 && cnt[tid]) atomicAdd(hist + tid, (unsigned long long)cnt[tid]);
}

// ------------------------------------------------------------------------------------------------ quality metrics

// max |x - y|, sum (x - y)^2, min x, max x.  The results are those of fp64 arithmetic, but the per-element work is
// done in fp32 with error-free transformations (fp64 instructions are an order of magnitude more expensive here):
// d = x - y together with its rounding error (the error is zero whenever x and y are within a factor of two of
// each other, which a reconstruction always is); d^2 as an exact fp32 pair (product and fused-multiply-add
// residual); the sum as a compensated fp32 pair.  A group of elements in which some difference is not an fp32
// number takes the fp64 path.  128-bit loads, per-thread accumulators, warp shuffles, one partial per CTA, and the
// last CTA to finish combines the partials in CTA order and writes the six results.
__global__ void __launch_bounds__(256, 4) quality_kernel(const float* __restrict__ x, const float* __restrict__ y, unsigned long long n,
                                                      double* __restrict__ out, double* __restrict__ partials, uint32_t* counter)
{
    pdl_enter();
    __shared__ double red[4][8];
    __shared__ uint32_t is_last;
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    float lo = __int_as_float(0x7F800000), hi = __int_as_float(0xFF800000), emax = 0.0f;
    // compensated sums of squares of the differences that are fp32 numbers: eight independent ones (one per element
    // of the two 128-bit loads in flight), so that consecutive elements do not wait for each other's additions
    float sh8[8] = {0.f, 0.f, 0.f, 0.f, 0.f, 0.f, 0.f, 0.f}, sl8[8] = {0.f, 0.f, 0.f, 0.f, 0.f, 0.f, 0.f, 0.f};
    double dmax = 0.0, dsum = 0.0;  // the others
    auto take = [&](float a, float b, int k) {
        float& sh = sh8[k];
        float& sl = sl8[k];
        lo = fminf(lo, a);
        hi = fmaxf(hi, a);
        const float d = __fsub_rn(a, b);
        const float bb = __fsub_rn(d, a);                                                     // TwoSum of a and -b
        const float err = __fsub_rn(__fsub_rn(a, __fsub_rn(d, bb)), __fadd_rn(b, bb));
        if (err == 0.0f) {
            emax = fmaxf(emax, fabsf(d));
            const float p = __fmul_rn(d, d), e = __fmaf_rn(d, d, -p);                         // d * d = p + e exactly
            const float t = __fadd_rn(sh, p), z = __fsub_rn(t, sh);
            sl = __fadd_rn(sl, __fadd_rn(__fadd_rn(__fsub_rn(sh, __fsub_rn(t, z)), __fsub_rn(p, z)), e));
            sh = t;
        } else {
            const double dd = (double)a - (double)b;
            dmax = fmax(dmax, fabs(dd));
            dsum += dd * dd;
        }
    };
    // The same arithmetic on two elements at a time (sm_100's packed fp32: each half rounds as the scalar operation
    // does), for the pairs of sums 2 k and 2 k + 1; a pair in which a difference is not an fp32 number goes element by
    // element.
    auto neg2 = [](float2 v) { return make_float2(-v.x, -v.y); };
    auto take2 = [&](float2 a, float2 b, int k) {
        const float2 d = __fadd2_rn(a, neg2(b));
        const float2 bb = __fadd2_rn(d, neg2(a));
        const float2 err = __fadd2_rn(__fadd2_rn(a, neg2(__fadd2_rn(d, neg2(bb)))), neg2(__fadd2_rn(b, bb)));
        if (err.x == 0.0f && err.y == 0.0f) {
            lo = fminf(lo, fminf(a.x, a.y));
            hi = fmaxf(hi, fmaxf(a.x, a.y));
            emax = fmaxf(emax, fmaxf(fabsf(d.x), fabsf(d.y)));
            const float2 shp = make_float2(sh8[2 * k], sh8[2 * k + 1]), slp = make_float2(sl8[2 * k], sl8[2 * k + 1]);
            const float2 p = __fmul2_rn(d, d), e = __ffma2_rn(d, d, neg2(p));
            const float2 t = __fadd2_rn(shp, p), z = __fadd2_rn(t, neg2(shp));
            const float2 r2 = __fadd2_rn(shp, neg2(__fadd2_rn(t, neg2(z)))), r3 = __fadd2_rn(p, neg2(z));
            const float2 sln = __fadd2_rn(slp, __fadd2_rn(__fadd2_rn(r2, r3), e));
            sh8[2 * k] = t.x; sh8[2 * k + 1] = t.y;
            sl8[2 * k] = sln.x; sl8[2 * k + 1] = sln.y;
        } else {
            take(a.x, b.x, 2 * k);
            take(a.y, b.y, 2 * k + 1);
        }
    };
    const unsigned long long gtid = (unsigned long long)blockIdx.x * blockDim.x + tid;
    const unsigned long long nth = (unsigned long long)gridDim.x * blockDim.x;
    unsigned long long done = 0;
    if (((((uintptr_t)x) | ((uintptr_t)y)) & 15u) == 0) {
        const unsigned long long nv = n >> 2;
        const float4* x4 = reinterpret_cast<const float4*>(x);
        const float4* y4 = reinterpret_cast<const float4*>(y);
        unsigned long long i = gtid;
        for (; i + nth < nv; i += 2 * nth) {   // two independent pairs of loads in flight
            const float4 a0 = __ldg(x4 + i), b0 = __ldg(y4 + i), a1 = __ldg(x4 + i + nth), b1 = __ldg(y4 + i + nth);
            take2(make_float2(a0.x, a0.y), make_float2(b0.x, b0.y), 0); take2(make_float2(a0.z, a0.w), make_float2(b0.z, b0.w), 1);
            take2(make_float2(a1.x, a1.y), make_float2(b1.x, b1.y), 2); take2(make_float2(a1.z, a1.w), make_float2(b1.z, b1.w), 3);
        }
        for (; i < nv; i += nth) {
            const float4 a = __ldg(x4 + i), b = __ldg(y4 + i);
            take(a.x, b.x, 0); take(a.y, b.y, 1); take(a.z, b.z, 2); take(a.w, b.w, 3);
        }
        done = nv << 2;
    }
    for (unsigned long long i = done + gtid; i < n; i += nth) take(__ldg(x + i), __ldg(y + i), 0);
    double sumsq = dsum;
#pragma unroll
    for (int k = 0; k < 8; ++k) sumsq += (double)sh8[k] + (double)sl8[k];   // fixed order
    double maxerr = fmax(dmax, (double)emax);
    double dlo = (double)lo, dhi = (double)hi;
#pragma unroll
    for (int d = 16; d >= 1; d >>= 1) {
        maxerr = fmax(maxerr, __shfl_xor_sync(kFull, maxerr, d));
        sumsq += __shfl_xor_sync(kFull, sumsq, d);
        dlo = fmin(dlo, __shfl_xor_sync(kFull, dlo, d));
        dhi = fmax(dhi, __shfl_xor_sync(kFull, dhi, d));
    }
    if (lane == 0) { red[0][warp] = maxerr; red[1][warp] = sumsq; red[2][warp] = dlo; red[3][warp] = dhi; }
    __syncthreads();
    if (tid == 0) {
        for (int w = 1; w < 8; ++w) {
            maxerr = fmax(maxerr, red[0][w]); sumsq += red[1][w]; dlo = fmin(dlo, red[2][w]); dhi = fmax(dhi, red[3][w]);
        }
        double* mine = partials + 4ull * blockIdx.x;
        mine[0] = maxerr; mine[1] = sumsq; mine[2] = dlo; mine[3] = dhi;
        __threadfence();
        is_last = atomicAdd(counter, 1u) == gridDim.x - 1 ? 1u : 0u;
    }
    __syncthreads();
    if (!is_last) return;
    // the last CTA: every thread takes the partials of CTAs tid, tid + 256, ... in that order, then the same tree as
    // above: a fixed order of additions whatever order the CTAs finished in
    __threadfence();
    maxerr = 0.0; sumsq = 0.0; dlo = __longlong_as_double(0x7FF0000000000000ll); dhi = __longlong_as_double(0xFFF0000000000000ull);
    for (unsigned b = tid; b < gridDim.x; b += 256) {
        const volatile double* pb = partials + 4ull * b;
        maxerr = fmax(maxerr, pb[0]); sumsq += pb[1]; dlo = fmin(dlo, pb[2]); dhi = fmax(dhi, pb[3]);
    }
#pragma unroll
    for (int d = 16; d >= 1; d >>= 1) {
        maxerr = fmax(maxerr, __shfl_xor_sync(kFull, maxerr, d));
        sumsq += __shfl_xor_sync(kFull, sumsq, d);
        dlo = fmin(dlo, __shfl_xor_sync(kFull, dlo, d));
        dhi = fmax(dhi, __shfl_xor_sync(kFull, dhi, d));
    }
    __syncthreads();   // the first round's values in `red` have been read
    if (lane == 0) { red[0][warp] = maxerr; red[1][warp] = sumsq; red[2][warp] = dlo; red[3][warp] = dhi; }
    __syncthreads();
    if (tid == 0) {
        for (int w = 1; w < 8; ++w) {
            maxerr = fmax(maxerr, red[0][w]); sumsq += red[1][w]; dlo = fmin(dlo, red[2][w]); dhi = fmax(dhi, red[3][w]);
        }
        const double mse = sumsq / (double)n, range = dhi - dlo;
        out[0] = maxerr; out[1] = mse; out[4] = dlo; out[5] = dhi;
        if (range > 0.0) {
            out[2] = sqrt(mse) / range;
            out[3] = mse > 0.0 ? 20.0 * log10(range / sqrt(mse)) : __longlong_as_double(0x7FF0000000000000ll);
        } else {
            out[2] = __longlong_as_double(0x7FF8000000000000ll);
            out[3] = __longlong_as_double(0x7FF8000000000000ll);
        }
        *counter = 0;
    }
}

std::atomic<unsigned long long> g_launches{0};   // kernels launched by this library in this process

}  // namespace

// ------------------------------------------------------------------------------------------------ launchers

unsigned long long launch_count() { return g_launches; }
void count_launches(unsigned k) { g_launches += k; }

cudaError_t launch_range(const RangeBatch& rb, const Workspace& ws, int sm_count, cudaStream_t st)
{
    if (rb.count <= 0) return cudaSuccess;
    unsigned long long nmax = 0;
    for (int j = 0; j < rb.count; ++j) nmax = rb.n[j] > nmax ? rb.n[j] : nmax;
    unsigned long long want = (nmax / 4 + 255) / 256;
    unsigned per = (unsigned)((sm_count * 8 + rb.count - 1) / rb.count);
    unsigned gx = (unsigned)(want < per ? (want ? want : 1) : per);
    ++g_launches;
    return launch_k(range_kernel, dim3(gx, rb.count), dim3(256), 0, st, rb, ws);
}

cudaError_t launch_encode(const JobBatch& jb, EncodeMode mode, const Workspace& ws, bool device_params,
                          Params host_params, int sm_count, cudaStream_t st)
{
    if (jb.total_tiles == 0) return cudaSuccess;
    if (mode == kEncodeRaw) {
        g_launches += (ws.slots && ws.skip_publish == 0xFFFFFFFFu) ? 2 : 1;
        return launch_encode_lanes(jb, ws, device_params, host_params, sm_count, st);
    }
    if (!ws.slots) return cudaErrorInvalidValue;   // the hop needs the slots of the two-step path
    g_launches += 2;
    return launch_hop_lanes(jb, ws, sm_count, st);
}

cudaError_t launch_decode(const JobBatch& jb, const Workspace& ws, int sm_count, cudaStream_t st)
{
    if (jb.total_tiles == 0) return cudaSuccess;
    ++g_launches;
    return launch_decode_lanes(jb, ws, sm_count, st);
}

cudaError_t launch_decode_wide(const DecodeBatch& jb, const Workspace& ws, int sm_count, cudaStream_t st)
{
    if (jb.total_tiles == 0) return cudaSuccess;
    ++g_launches;
    return launch_decode_lanes_wide(jb, ws, sm_count, st);
}

cudaError_t launch_copy(const CopyBatch& cb, const Workspace& ws, int sm_count, cudaStream_t st)
{
    if (cb.count <= 0) return cudaSuccess;
    unsigned gx = (unsigned)((sm_count * 4 + cb.count - 1) / cb.count);
    ++g_launches;
    return launch_k(copy_kernel, dim3(gx ? gx : 1, cb.count), dim3(256), 0, st, cb, ws);
}

cudaError_t launch_resolve_range(const float* minmax, float eb, const Workspace& ws, float* eb_abs_out, cudaStream_t st)
{
    ++g_launches;
    return launch_k(resolve_range_kernel, dim3(1), dim3(32), 0, st, minmax, eb, ws, eb_abs_out);
}

cudaError_t launch_scale(const ScaleBatch& sb, int sm_count, cudaStream_t st)
{
    if (sb.count <= 0 || sb.n == 0) return cudaSuccess;
    unsigned long long want = (sb.n + 255) / 256;
    unsigned per = (unsigned)((sm_count * 8 + sb.count - 1) / sb.count);
    unsigned gx = (unsigned)(want < per ? want : per);
    ++g_launches;
    return launch_k(scale_kernel, dim3(gx ? gx : 1, sb.count), dim3(256), 0, st, sb);
}

cudaError_t launch_quality(const float* x, const float* y, unsigned long long n, double* out, double* partials,
                           uint32_t* counter, int sm_count, cudaStream_t st)
{
    unsigned long long want = (n / 4 + 255) / 256;
    // one wave of resident CTAs, each striding over the arrays; asked of the current device on every call (a host-side
    // computation, no state shared between threads or devices)
    int per_sm = 0;
    if (cudaOccupancyMaxActiveBlocksPerMultiprocessor(&per_sm, quality_kernel, 256, 0) != cudaSuccess || per_sm < 1) per_sm = 1;
    unsigned long long cap = (unsigned long long)sm_count * per_sm;
    if (cap > (unsigned long long)kQualityCtas) cap = kQualityCtas;
    const unsigned grid = (unsigned)(want < cap ? (want ? want : 1) : cap);
    ++g_launches;
    return launch_k(quality_kernel, dim3(grid), dim3(256), 0, st, x, y, n, out, partials, counter);
}

cudaError_t launch_stream_stats(const uint32_t* in, unsigned long long cap_bytes, unsigned long long* hist, const Workspace& ws,
                                int sm_count, cudaStream_t st)
{
    ++g_launches;
    return launch_k(stream_stats_kernel, dim3((unsigned)sm_count * 2), dim3(256), 0, st, in, cap_bytes, hist, ws);
}

cudaError_t launch_copy_chain(const ChainBatch& cb, const Workspace& ws, int sm_count, cudaStream_t st, const CopyBatch* extra)
{
    static const CopyBatch none{};
    const int more = extra ? extra->count : 0;
    if ((cb.count <= 0 || cb.hops == 0) && more == 0) return cudaSuccess;
    ChainBatch chains = cb;
    if (cb.hops == 0) chains.count = 0;
    const int rows = chains.count + more;
    unsigned gx = (unsigned)((sm_count * 4 + rows - 1) / rows);
    ++g_launches;
    return launch_k(copy_chain_kernel, dim3(gx ? gx : 1, rows), dim3(256), 0, st, chains, extra ? *extra : none, ws);
}

}  // namespace zccl
