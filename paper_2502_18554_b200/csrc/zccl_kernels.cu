// fZ-light codec kernels for sm_100a: range reduction, bound resolution, encoder (plain and fused with a
// decode + add front end), decoder, and compressed-chunk copy.
//
// Work decomposition.  One CTA of 256 threads handles one 4096-element tile at a time; each of its 8 warps owns
// 16 consecutive 32-element blocks, one element per lane, so that a block's code length is one warp OR-reduction
// and its bit planes come out of a 32 x 32 bit-matrix transpose across the warp (one transpose serves four blocks
// while their code lengths fit 7 bits).  The kernels are bound by instruction issue (integer ALU pipe:
// 2 warp-instructions/clk/SM; shared memory and shuffles: 1) and by the latency of each tile's chain of phases, not
// by HBM, so the design minimises instructions per block and keeps barriers and one-thread work off that chain:
//   * tiles (encoder) and compressed blobs (decoder, fused hop) are staged in shared memory by 1-D bulk copies
//     (cp.async.bulk + mbarrier), requested one tile ahead, so no thread spends instructions or registers on
//     global loads and no warp waits on a chain of them;
//   * the common case runs in fp32 on the FMA pipe: codes are rounded with the 1.5*2^23 trick, deltas are float
//     subtractions (exact below 2^23), magnitudes are read from the mantissa of |delta| + 2^23.  Tiles whose
//     values leave the exactly representable range, ragged tails and unaligned inputs take an integer path
//     that computes the same bits;
//   * the encoder appends each block's words to its warp's region of shared memory in a single pass over the
//     block; the decoder undoes the Lorenzo recurrence by a warp-local transposition through shared memory
//     (16 consecutive elements per thread) instead of shuffle scans.
// The grid fits the device.  Decoder and fused hop deal tiles round-robin (CTA c takes tiles c, c + G, ...), so the
// next tiles are known in advance; the encoder hands them out in order through a device-wide counter, one tile
// ahead, so that a CTA which gets fewer issue slots takes fewer tiles.  Placement (prefix sum of tile sizes) is
// anchored at the tile a CTA placed last and deferred by one tile, so it only ever sums sizes that are already
// published; warp 0 plans a placement once for the CTA (layout, capacity check, index entry), warps 2..7 fetch the
// sizes for it, warp 1 requests the next tile meanwhile, and after one barrier every warp copies its own share.  The scan relies on the grid
// being resident at once; every wait is bounded and reports through the status word instead of hanging if it is
// not.
#include "zccl_device.cuh"

namespace zccl {

namespace {

constexpr int kSlotWords = 33;                 // sign word + up to 32 planes
constexpr int kBlobStageWords = 2048 + 8;      // compressed tiles up to 8 KiB are staged by bulk copy
constexpr int kFastDecodeMaxL = 18;


// Bit planes by a 32 x 32 bit-matrix transpose across the warp.  Lane j holds the word of element j (bit k =
// bit k of |delta_j|, bit 31 = its sign); after the transpose lane k holds plane k (bit j = that bit of element j)
// and lane 31 the sign word.  Five butterfly stages exchange bit-index bit b with lane-index bit b (b = 4..0): one
// shuffle plus a byte permute (strides 16, 8) or a rotate and a bit select (strides 4, 2, 1).  The transpose is
// its own inverse, so the decoder uses the same routine.  Cost does not depend on the code length, and there is no
// branch, so neighbouring blocks interleave.
struct Xpose {
    uint32_t sel16, sel8, m4, m2, m1, a4, a2, a1;
    __device__ __forceinline__ explicit Xpose(int lane)
    {
        sel16 = (lane & 16) ? 0x3276u : 0x5410u;
        sel8 = (lane & 8) ? 0x3715u : 0x6240u;
        m4 = (lane & 4) ? 0xF0F0F0F0u : 0x0F0F0F0Fu;
        m2 = (lane & 2) ? 0xCCCCCCCCu : 0x33333333u;
        m1 = (lane & 1) ? 0xAAAAAAAAu : 0x55555555u;
        a4 = (lane & 4) ? 28u : 4u;
        a2 = (lane & 2) ? 30u : 2u;
        a1 = (lane & 1) ? 31u : 1u;
        // hide the values' origin from the compiler: it would otherwise recompute the selects at every use
        asm volatile("" : "+r"(sel16), "+r"(sel8), "+r"(m4), "+r"(m2), "+r"(m1), "+r"(a4), "+r"(a2), "+r"(a1));
    }
    __device__ __forceinline__ uint32_t operator()(uint32_t x) const
    {
        uint32_t y = __shfl_xor_sync(kFull, x, 16);
        x = __byte_perm(x, y, sel16);
        y = __shfl_xor_sync(kFull, x, 8);
        x = __byte_perm(x, y, sel8);
        y = __shfl_xor_sync(kFull, x, 4);
        x = (x & m4) | (__funnelshift_l(y, y, a4) & ~m4);
        y = __shfl_xor_sync(kFull, x, 2);
        x = (x & m2) | (__funnelshift_l(y, y, a2) & ~m2);
        y = __shfl_xor_sync(kFull, x, 1);
        x = (x & m1) | (__funnelshift_l(y, y, a1) & ~m1);
        return x;
    }
};


// Per-lane constants of the packed store: with four blocks per transpose lane 8u + b ends up with plane b of
// block u (b = 7: its sign word).
struct PackLane {
    uint32_t sh8;   // 8 * (lane / 8): position of this lane's block in a word of four per-block bytes
    uint32_t wp;    // word of the block's slot this lane stores: 0 = sign word, b + 1 = plane b
    __device__ __forceinline__ explicit PackLane(int lane)
    {
        sh8 = 8u * ((uint32_t)lane >> 3);
        wp = ((uint32_t)(lane & 7) + 1u) & 7u;
        asm volatile("" : "+r"(sh8), "+r"(wp));
    }
};


// ------------------------------------------------------------------------------------------------ range (REL)

// eb -> (eb_abs, s, r), the reading used throughout: eb_abs = eb * (max - min); step shrunk by 1 - 2^-6;
// r by one IEEE division.  Consumes and re-arms the min/max keys.  One thread.
__device__ void resolve_params(float eb, const Workspace& ws)
{
    Params p;
    p.valid = 1;
    const uint32_t kmin = *reinterpret_cast<volatile uint32_t*>(ws.minmax + 0);
    const uint32_t kmax = *reinterpret_cast<volatile uint32_t*>(ws.minmax + 1);
    float range = 0.0f;
    if (kmin <= kmax) range = __fsub_rn(key2f(kmax), key2f(kmin));
    if (!(range > 0.0f) || !isfinite(range)) p.valid = 0;
    const float ea = __fmul_rn(eb, range);
    ws.minmax[0] = 0xFFFFFFFFu;
    ws.minmax[1] = 0u;
    const float ebq = __fmul_rn(ea, 0.984375f);
    const float s = __fmul_rn(ebq, 2.0f);
    if (!(s > 0.0f) || !isfinite(s)) p.valid = 0;
    const float r = __fdiv_rn(1.0f, s);
    if (!isfinite(r)) p.valid = 0;
    p.eb_abs = ea; p.s = s; p.r = r;
    *ws.params = p;
    if (!p.valid) atomicOr(ws.status, kStDegenerate);
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


// ================================================================================================ DECODE SIDE

// What a tile's index entry and code-length bytes say.  Uniform over the CTA (every warp reads the same words).
struct TileDesc {
    const uint32_t* blob;     // global: outlier word, code-length words, payload
    uint32_t words;           // blob size
    uint32_t nb, padw, len;
    int32_t outlier;
    bool ok;                  // sizes consistent with the index
    bool fast;                // full tile whose codes stay exact in fp32 and whose blob fits the staging buffer
    uint32_t lw;              // this lane's code-length word (blocks 4*lane .. 4*lane+3)
    uint32_t o0, o1, o2, o3;  // payload offsets (words) of this lane's four blocks
};

__device__ __forceinline__ TileDesc describe_tile(const uint32_t* __restrict__ in, unsigned long long cap_bytes,
                                                  const StreamInfo& h, uint32_t tile, int lane)
{
    TileDesc d;
    d.ok = false; d.fast = false; d.blob = in; d.words = 0; d.outlier = 0; d.lw = 0; d.o0 = d.o1 = d.o2 = d.o3 = 0;
    const uint32_t* idx = in + kHeaderWords;
    const uint32_t w_end = ldg_u32(idx + tile);
    const uint32_t w_beg = tile ? ldg_u32(idx + tile - 1) : 0u;
    const unsigned long long blob0 = (unsigned long long)kHeaderWords + h.nT;   // in words
    const unsigned long long start = (unsigned long long)tile * kTile;
    d.len = (uint32_t)((h.n - start < (unsigned long long)kTile) ? (h.n - start) : kTile);
    d.nb = (d.len + kBlock - 1) / kBlock;
    d.padw = (d.nb + 3) >> 2;
    if (w_end < w_beg) return d;
    if ((blob0 + w_end) * 4ull > cap_bytes) return d;
    d.words = w_end - w_beg;
    if (d.words < 1 + d.padw) return d;
    d.blob = in + blob0 + w_beg;
    d.outlier = (int32_t)ldg_u32(d.blob);

    // code lengths: one word (4 blocks) per lane; sizes; warp-wide exclusive scan of the sizes
    const uint32_t lw = ((uint32_t)lane < d.padw) ? ldg_u32(d.blob + 1 + lane) : 0u;
    const uint32_t L0 = lw & 0xFF, L1 = (lw >> 8) & 0xFF, L2 = (lw >> 16) & 0xFF, L3 = lw >> 24;
    bool bad = (L0 > 31) | (L1 > 31) | (L2 > 31) | (L3 > 31);
    const uint32_t b0 = 4u * lane;   // blocks at or beyond nb are padding of the code-length area: must be zero
    if ((b0 + 0 >= d.nb && L0) || (b0 + 1 >= d.nb && L1) || (b0 + 2 >= d.nb && L2) || (b0 + 3 >= d.nb && L3)) bad = true;
    const uint32_t z0 = L0 ? L0 + 1 : 0, z1 = L1 ? L1 + 1 : 0, z2 = L2 ? L2 + 1 : 0, z3 = L3 ? L3 + 1 : 0;
    const uint32_t lane_sum = z0 + z1 + z2 + z3;
    uint32_t incl = lane_sum;
#pragma unroll
    for (int s = 1; s < 32; s <<= 1) {
        uint32_t t = __shfl_up_sync(kFull, incl, s);
        if (lane >= s) incl += t;
    }
    const uint32_t total = __shfl_sync(kFull, incl, 31);
    bad = __any_sync(kFull, bad);
    if (bad || 1 + d.padw + total != d.words) return d;
    d.ok = true;
    d.lw = lw;
    d.o0 = incl - lane_sum; d.o1 = d.o0 + z0; d.o2 = d.o1 + z1; d.o3 = d.o2 + z2;

    // fp32 exactness: every partial sum of deltas is below sum_b 32 * 2^L_b; with the outlier it must stay < 2^24
    const uint32_t Lmax = max(max(L0, L1), max(L2, L3));
    uint32_t spread = 1u << 24;
    if (Lmax <= (uint32_t)kFastDecodeMaxL) spread = (32u << L0) + (32u << L1) + (32u << L2) + (32u << L3);
    spread = __reduce_add_sync(kFull, min(spread, 1u << 24));   // at most 32 * 2^24 = 2^29: no overflow
    const uint32_t ao = (uint32_t)(d.outlier < 0 ? -d.outlier : d.outlier);
    const bool exact = ao < (1u << 23) && spread < (1u << 23);
    // staging copies the 16-byte-aligned cover of the blob; it must stay inside the readable bytes
    const uintptr_t a_beg = (uintptr_t)d.blob & ~(uintptr_t)15;
    const uintptr_t a_end = ((uintptr_t)(d.blob + d.words) + 15) & ~(uintptr_t)15;
    const bool stageable = (a_end - a_beg) <= (uintptr_t)(kBlobStageWords * 4) &&
                           (a_end - (uintptr_t)in) <= (uintptr_t)cap_bytes;
    d.fast = exact && stageable && d.len == (uint32_t)kTile;
    return d;
}

// Integer path: decodes this warp's 16 blocks straight from global memory into codes relative to the warp's first
// element, one element per lane (q[i] = sum of deltas from the warp's first element; the caller adds the outlier
// and the sums of the preceding warps).
__device__ __forceinline__ void decode_blocks_int(const TileDesc& d, int warp, int lane, int32_t* __restrict__ q)
{
    const uint32_t* payload = d.blob + 1 + d.padw;
    int32_t carry = 0;
#pragma unroll 1
    for (int i = 0; i < kBlocksPerWarp; ++i) {
        const int src = 4 * warp + (i >> 2);
        const uint32_t lwi = __shfl_sync(kFull, d.lw, src);
        const uint32_t L = (lwi >> (8 * (i & 3))) & 0xFF;
        const uint32_t osel = (i & 3) == 0 ? d.o0 : (i & 3) == 1 ? d.o1 : (i & 3) == 2 ? d.o2 : d.o3;
        const uint32_t off = __shfl_sync(kFull, osel, src);
        int32_t v = 0;
        if (L) {   // uniform over the warp
            const uint32_t word = ((uint32_t)lane <= L) ? ldg_u32(payload + off + lane) : 0u;
            const uint32_t sign = __shfl_sync(kFull, word, 0);
            uint32_t mag = 0;
            for (uint32_t k = 0; k < L; ++k) {
                const uint32_t plane = __shfl_sync(kFull, word, k + 1);
                mag |= ((plane >> lane) & 1u) << k;
            }
            v = ((sign >> lane) & 1u) ? -(int32_t)mag : (int32_t)mag;
#pragma unroll
            for (int s = 1; s < 32; s <<= 1) {
                int32_t t = __shfl_up_sync(kFull, v, s);
                if (lane >= s) v += t;
            }
        }
        q[i] = carry + v;
        carry = __shfl_sync(kFull, q[i], 31);
    }
}

// fp32 path: rebuilds this warp's 16 blocks of deltas from the staged blob and stores them, as exact floats, in
// the warp's 512-word region `wbuf`, row i = block i, element j of a row at word j ^ ((i & 3) << 2) (so that the
// 128-bit reads of decode_scan_f32 are free of bank conflicts).  tbl: per block {code length, payload address}.
// UNROLL: the fused hop unrolls the loop over the groups of four completely (fewer instructions, 75 -> 73 us); the
// decoder, at its 48 registers, is fastest with two groups per iteration (35.2 -> 34.4 us; 35.2 again with four).
template <int UNROLL>
__device__ __forceinline__ void decode_blocks_f32(const uint2* __restrict__ tbl, float* __restrict__ wbuf, int lane,
                                                  const Xpose& xp)
{
    const uint32_t widx = (uint32_t)(lane + 1) & 31u;   // lane k fetches plane k (word k + 1), lane 31 the sign word
    const PackLane pk(lane);
    const uint2* my_tbl = tbl + (lane >> 3);
#pragma unroll UNROLL
    for (int g = 0; g < kBlocksPerWarp / 4; ++g) {
        const uint2 em = my_tbl[4 * g];           // entry of block 4g + lane / 8: code length, shared address of the payload
        if (!__any_sync(kFull, em.x > 7u)) {
            // four blocks per transpose: lane 8u + b fetches plane b of block u (b = 7: its sign word)
            const uint32_t n = em.x ? em.x + 1 : 0;
            uint32_t w = 0;
            if (pk.wp < n) asm volatile("ld.shared.u32 %0, [%1];" : "=r"(w) : "r"(em.y + 4 * pk.wp) : "memory");
            const uint32_t v = xp(w);             // byte u: bits 0..6 = |delta| of this lane's element of block u, bit 7 = sign
            const uint32_t vm = v & 0x7F7F7F7Fu;
#pragma unroll
            for (int u = 0; u < 4; ++u) {
                const int i = 4 * g + u;
                const float mag = __fsub_rn(__uint_as_float(prmt(vm, 0x4B000000u, 0x7540u | (uint32_t)u)), kTwo23);
                const uint32_t sg = prmt(v, v, (0x8u | (uint32_t)u) << 12);   // byte 3 = sign of byte u, replicated
                wbuf[32 * i + (lane ^ (u << 2))] = __uint_as_float(__float_as_uint(mag) | (sg & 0x80000000u));
            }
        } else if (!__any_sync(kFull, em.x > 15u)) {
            // two blocks per transpose: lane 16u + b fetches plane b of block 2h + u (b = 15: its sign word)
            const uint32_t wp2 = ((uint32_t)lane + 1u) & 15u;
#pragma unroll
            for (int h = 0; h < 2; ++h) {
                const uint2 e = tbl[4 * g + 2 * h + (lane >> 4)];
                const uint32_t n = e.x ? e.x + 1 : 0;
                uint32_t w = 0;
                if (wp2 < n) asm volatile("ld.shared.u32 %0, [%1];" : "=r"(w) : "r"(e.y + 4 * wp2) : "memory");
                const uint32_t v = xp(w);   // half u: bits 0..14 = |delta| of this lane's element of block 2h + u, bit 15 = sign
#pragma unroll
                for (int u = 0; u < 2; ++u) {
                    const int b4 = 2 * h + u, i = 4 * g + b4;
                    const uint32_t m = u ? (v >> 16) & 0x7FFFu : v & 0x7FFFu;
                    const float mag = __fsub_rn(__uint_as_float(m | 0x4B000000u), kTwo23);
                    const uint32_t sg = u ? v : v << 16;
                    wbuf[32 * i + (lane ^ (b4 << 2))] = __uint_as_float(__float_as_uint(mag) | (sg & 0x80000000u));
                }
            }
        } else {
#pragma unroll
            for (int u = 0; u < 4; ++u) {
                const int i = 4 * g + u;
                const uint2 e = tbl[i];           // broadcast read
                const uint32_t sz = e.x ? e.x + 1 : 0;
                uint32_t w = 0;
                if (widx < sz) asm volatile("ld.shared.u32 %0, [%1];" : "=r"(w) : "r"(e.y + 4 * widx) : "memory");
                const uint32_t v = xp(w);         // bits 0..L-1: |delta| of this lane's element, bit 31: its sign
                // exact fp32 value of the magnitude from its bits (|delta| < 2^23), then the sign bit on top
                const float mag = __fsub_rn(__uint_as_float((v & 0x007FFFFFu) | 0x4B000000u), kTwo23);
                wbuf[32 * i + (lane ^ (u << 2))] = __uint_as_float(__float_as_uint(mag) | (v & 0x80000000u));
            }
        }
    }
}

// Reads this thread's 16 consecutive deltas (elements 16*lane .. 16*lane+15 of the warp's 512) from `wbuf`,
// forms their running sum and the warp-wide exclusive prefix.  On return v[k] = sum of the warp's deltas up to
// and including this thread's element k; the return value is the warp's total.
// `excl` receives the sum of the warp's deltas before this thread's first element: v[k] is then only the running sum
// inside the thread, and the caller adds excl (plus whatever comes before the warp) once, in one addition per element.
__device__ __forceinline__ float decode_scan_f32(const float* __restrict__ wbuf, int lane, float (&v)[16], float& excl)
{
    const int sw = (lane >> 1) & 3;
    const float4* row = reinterpret_cast<const float4*>(wbuf + 16 * lane);
#pragma unroll
    for (int c = 0; c < 4; ++c) {
        const float4 f = row[c ^ sw];
        v[4 * c + 0] = f.x; v[4 * c + 1] = f.y; v[4 * c + 2] = f.z; v[4 * c + 3] = f.w;
    }
    float run = 0.0f;
#pragma unroll
    for (int k = 0; k < 16; ++k) { run = __fadd_rn(run, v[k]); v[k] = run; }
    float incl = run;
#pragma unroll
    for (int s = 1; s < 32; s <<= 1) {
        const float t = __shfl_up_sync(kFull, incl, s);
        if (lane >= s) incl = __fadd_rn(incl, t);
    }
    excl = __fsub_rn(incl, run);
    return __shfl_sync(kFull, incl, 31);
}

// Where a tile's blob is, as known from the index alone (no access to the blob itself).
struct BlobSpan {
    uint32_t w_beg, w_end;   // index entries: blob = words [w_beg, w_end) of the blob area
    uint32_t staged;         // 1: its 16-byte-aligned cover was requested by a bulk copy
};

// The 16-byte-aligned cover of a blob can be staged when it fits the staging buffer and lies inside the readable
// bytes of the stream.
__device__ __forceinline__ bool blob_stageable(const uint32_t* in, unsigned long long cap_bytes, uint32_t nT, uint32_t w_beg,
                                               uint32_t w_end, uintptr_t& a_beg, uint32_t& bytes)
{
    if (w_end <= w_beg) return false;
    const unsigned long long blob0 = (unsigned long long)kHeaderWords + nT;
    if ((blob0 + w_end) * 4ull > cap_bytes) return false;
    const uintptr_t b = (uintptr_t)(in + blob0 + w_beg), e = (uintptr_t)(in + blob0 + w_end);
    a_beg = b & ~(uintptr_t)15;
    const uintptr_t a_end = (e + 15) & ~(uintptr_t)15;
    bytes = (uint32_t)(a_end - a_beg);
    return (a_end - a_beg) <= (uintptr_t)(kBlobStageWords * 4) && (a_end - (uintptr_t)in) <= (uintptr_t)cap_bytes;
}

// Thread 0 of a CTA runs ahead of the others: it keeps the index entries of the tile after next in registers and
// turns the next tile's entries into a bulk copy of its blob, so that no warp waits on a chain of global loads.
// Shared needs: blob[2][kBlobStageWords], span[2], bar[2].
struct StagePipe {
    uint32_t n_beg = 0, n_end = 0;   // index entries of the next tile (valid when n_job >= 0)
    int n_job = -1;

    // index entries of tile number t of the launch
    __device__ __forceinline__ void fetch(const JobBatch& jb, uint32_t t, int cur_job, const StreamInfo& h, uint32_t limit = 0xFFFFFFFFu)
    {
        n_job = -1;
        if (t >= jb.total_tiles || t >= limit) return;   // limit: end of the CTA's own range of tiles
        const int jj = find_job(jb, t);
        const Job& jq = jb.job[jj];
        const uint32_t tl = t - jq.tile_begin;
        // the index entries do not depend on the header's contents, only on their being inside the readable bytes:
        // ask for them first, so that they travel together with the header instead of after it
        const uint32_t* idx = jq.in_c + kHeaderWords;
        const bool inside = ((unsigned long long)kHeaderWords + tl + 1ull) * 4ull <= jq.in_cap;
        const uint32_t e_end = inside ? ldg_u32(idx + tl) : 0u;
        const uint32_t e_beg = (inside && tl) ? ldg_u32(idx + tl - 1) : 0u;
        const StreamInfo hq = (jj == cur_job) ? h : read_header(jq.in_c, jq.in_cap);
        if (!hq.ok || hq.n > jq.n || tl >= hq.nT) return;   // a valid header guarantees that the whole index is readable
        n_end = e_end;
        n_beg = e_beg;
        n_job = jj;
    }
    // request the blob of tile t (whose entries were fetched before) into staging buffer `buf`
    template <class Shared>
    __device__ __forceinline__ void stage(Shared& sh, const JobBatch& jb, uint32_t t, int cur_job, const StreamInfo& h, uint32_t buf)
    {
        BlobSpan sp;
        sp.w_beg = n_beg; sp.w_end = n_end; sp.staged = 0;
        if (n_job >= 0) {
            const Job& jq = jb.job[n_job];
            const StreamInfo hq = (n_job == cur_job) ? h : read_header(jq.in_c, jq.in_cap);
            const uint32_t tl = t - jq.tile_begin;
            const unsigned long long start = (unsigned long long)tl * kTile;
            uintptr_t a_beg = 0;
            uint32_t bytes = 0;
            if (hq.ok && !jq.in_c2 && hq.n - start >= (unsigned long long)kTile &&
                blob_stageable(jq.in_c, jq.in_cap, hq.nT, n_beg, n_end, a_beg, bytes)) {
                mbar_expect_tx(&sh.bar[buf], bytes);
                bulk_load(sh.blob[buf], (const void*)a_beg, bytes, &sh.bar[buf]);
                sp.staged = 1;
                // the fused kernel adds a local operand to this tile: have it in L2 by then
                if (jq.x && (((uintptr_t)(jq.x + start)) & 15u) == 0) bulk_prefetch_l2(jq.x + start, kTile * 4);
            }
        }
        sh.span[buf] = sp;
    }
};

struct DecodeShared {
    alignas(16) uint32_t blob[2][kBlobStageWords];            // staged blobs: current tile and the next one
    alignas(16) float wbuf[kWarps][kBlocksPerWarp * kBlock];
    alignas(16) uint2 tbl[kBlocksPerTile];                    // per block {code length, shared address of its payload}
    BlobSpan span[2];
    float warp_total[2][kWarps];
    int32_t warp_total_i[kWarps];
    alignas(8) unsigned long long bar[2];
};

// Description of a staged full tile, by every warp on its own (no barrier): lane l reads the code lengths of blocks
// 4l .. 4l+3, a warp-wide scan gives every block's payload offset, and the lanes that hold the warp's own 16 blocks
// write their entries of the block table {code length, shared address of the payload}.  Checks the code lengths
// against the blob size and decides whether the tile's codes stay exact in fp32.  Every warp reaches the same
// verdict.  Returns 0: inconsistent blob, 1: take the fp32 path, 2: consistent but needs the integer path.
__device__ __forceinline__ int describe_staged(uint2* __restrict__ tbl, const uint32_t* sb, uint32_t words, int lane, int warp)
{
    constexpr uint32_t padw = kBlocksPerTile / 4;
    const uint32_t lw = sb[1 + lane];
    const uint32_t L0 = lw & 0xFFu, L1 = (lw >> 8) & 0xFFu, L2 = (lw >> 16) & 0xFFu, L3 = lw >> 24;
    const bool bad = ((lw & 0xE0E0E0E0u) != 0u);   // a code length above 31
    const uint32_t z0 = L0 ? L0 + 1 : 0, z1 = L1 ? L1 + 1 : 0, z2 = L2 ? L2 + 1 : 0, z3 = L3 ? L3 + 1 : 0;
    const uint32_t lane_sum = z0 + z1 + z2 + z3;
    uint32_t incl = lane_sum;
#pragma unroll
    for (int d = 1; d < 32; d <<= 1) {
        const uint32_t t = __shfl_up_sync(kFull, incl, d);
        if (lane >= d) incl += t;
    }
    const uint32_t total = __shfl_sync(kFull, incl, 31);
    const uint32_t Lmax = max(max(L0, L1), max(L2, L3));
    uint32_t spread = 1u << 24;
    if (Lmax <= (uint32_t)kFastDecodeMaxL) spread = (32u << L0) + (32u << L1) + (32u << L2) + (32u << L3);
    spread = __reduce_add_sync(kFull, min(spread, 1u << 24));   // at most 32 * 2^24 = 2^29: no overflow
    if (__any_sync(kFull, bad) || 1 + padw + total != words) return 0;
    if ((lane >> 2) == warp) {   // this lane's four blocks are blocks 4 (lane & 3) .. of the warp
        const uint32_t a0 = smem_u32(sb + 1 + padw) + 4 * (incl - lane_sum);
        uint2* e = tbl + kBlocksPerWarp * warp + 4 * (lane & 3);
        e[0] = make_uint2(L0, a0);
        e[1] = make_uint2(L1, a0 + 4 * z0);
        e[2] = make_uint2(L2, a0 + 4 * (z0 + z1));
        e[3] = make_uint2(L3, a0 + 4 * (z0 + z1 + z2));
    }
    __syncwarp();
    const int32_t outlier = (int32_t)sb[0];
    const uint32_t ao = (uint32_t)(outlier < 0 ? -outlier : outlier);
    return (ao < (1u << 23) && spread < (1u << 23)) ? 1 : 2;
}

__global__ void __launch_bounds__(kThreads, 5) decode_kernel(JobBatch jb, Workspace ws)
{
    pdl_enter();
    __shared__ DecodeShared sh;
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    // every CTA takes a run of consecutive tiles: their blobs and index entries are neighbours in the stream, and in a
    // launch of many short jobs (the chunks of a ring) a CTA stays inside one job instead of changing it with every tile
    // (the first `rem` CTAs take one tile more than the others, as dealing them round-robin would give them)
    const uint32_t quo = jb.total_tiles / gridDim.x, rem = jb.total_tiles % gridDim.x;
    const uint32_t g0 = blockIdx.x * quo + (blockIdx.x < rem ? blockIdx.x : rem);
    const uint32_t g1 = g0 + quo + (blockIdx.x < rem ? 1u : 0u);
    uint32_t status = 0;
    uint32_t fills0 = 0, fills1 = 0;   // bulk copies completed per staging buffer (phase parity of its mbarrier)
    uint32_t par = 0;                  // parity of the warp_total double buffer
    uint32_t p = 0;                    // staging buffer of the current tile
    const Xpose xp(lane);

    int cur_job = -1;
    StreamInfo h;
    h.ok = false; h.n = 0; h.nT = 0; h.s = 1.0f; h.eb_abs = 0.0f;

    StagePipe pipe;   // thread 0 only
    if (tid == 0) {
        mbar_init(&sh.bar[0], 1);
        mbar_init(&sh.bar[1], 1);
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
        pipe.fetch(jb, g0, cur_job, h, g1);
        pipe.stage(sh, jb, g0, cur_job, h, 0);
        pipe.fetch(jb, g0 + 1, cur_job, h, g1);
    }
    __syncthreads();

    for (uint32_t g = g0; g < g1; ++g) {
        const int j = find_job(jb, g);
        const Job& job = jb.job[j];
        if (j != cur_job) { h = read_header(job.in_c, job.in_cap); cur_job = j; }
        const uint32_t tile = g - job.tile_begin;

        // thread 0: request the next tile's blob into the other buffer (its readers finished before the last barrier
        // of the previous iteration), then fetch the index entries of the tile after it
        if (tid == 0) {
            pipe.stage(sh, jb, g + 1, cur_job, h, p ^ 1u);
            pipe.fetch(jb, g + 2, cur_job, h, g1);
        }
        const BlobSpan sp = sh.span[p];
        if (sp.staged) {   // a copy was requested for this tile: always consume it, whatever happens next
            const uint32_t fl = p ? fills1 : fills0;
            if (!mbar_wait(&sh.bar[p], fl & 1u)) status |= kStTimeout;
            if (p) ++fills1; else ++fills0;
        }
        bool skip_tile = false;
        if (!h.ok) { status |= kStBadStream; skip_tile = true; }
        else if (h.n > job.n) { status |= kStCapacity; skip_tile = true; }
        else if (tile >= h.nT) skip_tile = true;

        int mode = 2;   // 1: fp32 path from the staged blob, 2: integer path from global memory
        if (!skip_tile && sp.staged) {
            const unsigned long long blob0 = (unsigned long long)kHeaderWords + h.nT;
            const uint32_t shift = (uint32_t)(((uintptr_t)(job.in_c + blob0 + sp.w_beg) & 15u) >> 2);
            const uint32_t* sb = sh.blob[p] + shift;
            mode = describe_staged(sh.tbl, sb, sp.w_end - sp.w_beg, lane, warp);
            if (mode == 0) { status |= kStBadStream; skip_tile = true; }
            if (mode == 1) {
                float* __restrict__ y = job.y + (unsigned long long)tile * kTile;
                decode_blocks_f32<2>(sh.tbl + kBlocksPerWarp * warp, sh.wbuf[warp], lane, xp);
                __syncwarp();
                float v[16];
                float before;
                const float total = decode_scan_f32(sh.wbuf[warp], lane, v, before);
                if (lane == 0) sh.warp_total[par][warp] = total;
                const float outlier = (float)(int32_t)sb[0];
                __syncthreads();
                float base = outlier;
                for (int w = 0; w < warp; ++w) base = __fadd_rn(base, sh.warp_total[par][w]);
                base = __fadd_rn(base, before);   // all of these are integers below 2^24: any order of addition is exact
                par ^= 1u;
                // A thread holds 16 consecutive elements; stored from there, a 128-bit store would touch 32 separate
                // 64-byte pieces and be replayed.  The values go back through the warp's rows instead (same swizzle as
                // the deltas), so that store c of the warp writes 512 consecutive bytes.
                float4* wrow = reinterpret_cast<float4*>(sh.wbuf[warp]);
                const int sw = (lane >> 1) & 3;
#pragma unroll
                for (int c = 0; c < 4; ++c) {
                    float4 o;
                    o.x = __fmul_rn(__fadd_rn(v[4 * c + 0], base), h.s);
                    o.y = __fmul_rn(__fadd_rn(v[4 * c + 1], base), h.s);
                    o.z = __fmul_rn(__fadd_rn(v[4 * c + 2], base), h.s);
                    o.w = __fmul_rn(__fadd_rn(v[4 * c + 3], base), h.s);
                    wrow[4 * lane + (c ^ sw)] = o;
                }
                __syncwarp();
                float4* dst = reinterpret_cast<float4*>(y + 512 * warp);
                const bool vec = (((uintptr_t)dst) & 15u) == 0;
#pragma unroll
                for (int c = 0; c < 4; ++c) {
                    const int f = 32 * c + lane, t = f >> 2;           // float4 number f of the warp's 128: thread t's
                    const float4 o = wrow[4 * t + ((f & 3) ^ ((t >> 1) & 3))];
                    if (vec) dst[f] = o;
                    else {
                        float* ds = reinterpret_cast<float*>(dst + f);
                        ds[0] = o.x; ds[1] = o.y; ds[2] = o.z; ds[3] = o.w;
                    }
                }
            }
        }
        if (!skip_tile && mode == 2) {
            const TileDesc d = describe_tile(job.in_c, job.in_cap, h, tile, lane);
            if (!d.ok) status |= kStBadStream;
            else {
                float* __restrict__ y = job.y + (unsigned long long)tile * kTile;
                int32_t q[kBlocksPerWarp];
                decode_blocks_int(d, warp, lane, q);
                __syncthreads();
                if (lane == 31) sh.warp_total_i[warp] = q[kBlocksPerWarp - 1];
                __syncthreads();
                int32_t base = d.outlier;
                for (int w = 0; w < warp; ++w) base += sh.warp_total_i[w];
                const uint32_t e0 = (uint32_t)(warp * kBlocksPerWarp * kBlock + lane);
#pragma unroll
                for (int i = 0; i < kBlocksPerWarp; ++i) {
                    const uint32_t e = e0 + (uint32_t)(i * kBlock);
                    if (e < d.len) y[e] = __fmul_rn(__int2float_rn(base + q[i]), h.s);
                }
            }
        }
        __syncthreads();   // keeps the warps of a CTA in step (measured faster than letting them drift apart)
        p ^= 1u;
    }
    // a copy requested for a tile beyond the last one is never started (stage_span checks the tile number); after an
    // expired wait give the outstanding copies one more bounded wait before leaving
    if (tid == 0 && (status & kStTimeout)) {
        (void)mbar_wait(&sh.bar[0], (fills0 + 1u) & 1u);
        (void)mbar_wait(&sh.bar[1], (fills1 + 1u) & 1u);
    }
    if (status) atomicOr(ws.status, status);
}

// ================================================================================================ ENCODE SIDE

// Where a warp reads the values it encodes.  cur(g, u) / prev(g, u): element `lane` of the warp's block 4g + u
// and the element before it (the tile's first element is its own predecessor: its delta is zero by definition).
struct SrcStaged {          // tile staged in shared memory in element order, with one guard word in front
    const float* xb;        // &tile[512 * warp + lane]
    __device__ __forceinline__ float cur(int g, int u) const { return xb[32 * (4 * g + u)]; }
    __device__ __forceinline__ float prev(int g, int u) const { return xb[32 * (4 * g + u) - 1]; }
};
struct SrcGlobal {          // straight from global memory, any alignment, ragged tails repeat the last element
    const float* x;         // tile start
    uint32_t e0;            // 512 * warp + lane
    uint32_t last;          // len - 1
    __device__ __forceinline__ float cur(int g, int u) const
    {
        const uint32_t e = e0 + 32u * (4 * g + u);
        return __ldg(x + (e < last ? e : last));
    }
    __device__ __forceinline__ float prev(int g, int u) const
    {
        const uint32_t e = e0 + 32u * (4 * g + u);
        const uint32_t ep = e ? e - 1 : 0;
        return __ldg(x + (ep < last ? ep : last));
    }
};
struct SrcSwizzled {        // the fused kernel's sum tile: per-warp region of 17 rows (row 0 = guard row); element j
    const float* rows;      // of block i lives at rows[32 * (i + 1) + (j ^ ((i & 3) << 2))]
    int co[4];              // lane's word within a row of block 4g + u
    int po[4];              // predecessor's word relative to the same row (lane 0: last element of the row before)
    __device__ __forceinline__ SrcSwizzled(const float* r, int lane) : rows(r)
    {
#pragma unroll
        for (int u = 0; u < 4; ++u) {
            co[u] = lane ^ (u << 2);
            po[u] = lane ? ((lane - 1) ^ (u << 2)) : (-32 + (31 ^ (((u + 3) & 3) << 2)));
        }
    }
    __device__ __forceinline__ float cur(int g, int u) const { return rows[32 * (4 * g + u + 1) + co[u]]; }
    __device__ __forceinline__ float prev(int g, int u) const { return rows[32 * (4 * g + u + 1) + po[u]]; }
};

// One pass over this warp's 16 blocks: quantise, 1-D Lorenzo delta, code length, sign word and bit planes, appended
// to the warp's region of shared memory.  Returns the warp's payload size in words; lane g (g < 4) ends up holding
// the code-length word of blocks 4g..4g+3 in `my_lw`.  FAST: fp32 arithmetic, valid while every |x * r| < 2^21.5;
// the caller checks `guard` (sum of squares of x * r over the warp's elements and the one before them) and reruns
// with FAST = false when it is too large.  FAST handles four blocks per bit-matrix transpose while their code
// lengths are at most 7 (sign + 7 magnitude bits of four elements share a word), else one block per transpose.
template <bool FAST, int UNROLL = 4, class Src>
__device__ __forceinline__ uint32_t encode_blocks(const Src& src, float r, uint32_t* __restrict__ slots_w, int lane,
                                                  const Xpose& xp, uint32_t& my_lw, float& guard, float& tmax)
{
    uint32_t wsum = 0;
    float acc = 0.0f, tm = 0.0f;
    my_lw = 0;
    const uint32_t widx = (uint32_t)(lane + 1) & 31u;   // lane k stores plane k at word k + 1, lane 31 the sign word at 0
    const PackLane pk(lane);
    if (FAST) {   // the element before the warp's first one belongs to nobody else's sum
        const float tp0 = __fmul_rn(src.prev(0, 0), r);
        if (lane == 0) acc = __fmul_rn(tp0, tp0);
    }
#pragma unroll UNROLL
    for (int g = 0; g < kBlocksPerWarp / 4; ++g) {   // unrolled by default: constant offsets, 5 % fewer instructions
        uint32_t lword = 0;
        if (FAST) {
            uint32_t ab[4], db[4];
#pragma unroll
            for (int u = 0; u < 4; ++u) {
                const float t = __fmul_rn(src.cur(g, u), r), tp = __fmul_rn(src.prev(g, u), r);
                acc = __fmaf_rn(t, t, acc);
                const float df = __fsub_rn(__fadd_rn(t, kRoundMagic), __fadd_rn(tp, kRoundMagic));
                // magnitude in bits 0..22 (bits 23..30 hold exponent bits: never stored, L <= 23)
                ab[u] = __float_as_uint(__fadd_rn(fabsf(df), kTwo23));
                db[u] = __float_as_uint(df);
            }
            const uint32_t wide = ((ab[0] | ab[1] | ab[2]) | ab[3]) & 0x7FFF80u;   // magnitude bits above bit 6
            if (!__any_sync(kFull, wide != 0)) {
                // byte u of the word: bits 0..6 = |delta| of this lane's element of block u, bit 7 = its sign
                const uint32_t mg = prmt(prmt(ab[0], ab[1], 0x0040u), prmt(ab[2], ab[3], 0x0040u), 0x5410u);
                const uint32_t sg = prmt(prmt(db[0], db[1], 0x00FBu), prmt(db[2], db[3], 0x00FBu), 0x5410u);
                const uint32_t v = xp(mg | (sg & 0x80808080u));
                const uint32_t ors = __reduce_or_sync(kFull, mg);                       // byte u: OR of block u's magnitudes
                const uint32_t l_mine = 32u - (uint32_t)__clz((int)((ors >> pk.sh8) & 0xFFu));
                lword = __reduce_or_sync(kFull, l_mine << pk.sh8);                      // byte u: code length of block u
                const uint32_t nword = lword + (((lword + 0x7F7F7F7Fu) >> 7) & 0x01010101u);   // byte u: slot size of block u
                const uint32_t pref = nword * 0x01010100u;                              // byte u: slots of blocks before u
                const uint32_t n_mine = (nword >> pk.sh8) & 0xFFu;
                if (pk.wp < n_mine) slots_w[wsum + ((pref >> pk.sh8) & 0xFFu) + pk.wp] = v;
                wsum += (nword * 0x01010101u) >> 24;
            } else if (!__any_sync(kFull, (wide & 0x7F8000u) != 0)) {
                // two blocks per transpose while their code lengths are at most 15: half u of the word holds
                // |delta| of this lane's element of block 2h + u in bits 0..14 and its sign in bit 15, so lane
                // 16u + b ends up with plane b of that block (b = 15: its sign word)
#pragma unroll
                for (int h = 0; h < 2; ++h) {
                    const uint32_t mg = prmt(ab[2 * h], ab[2 * h + 1], 0x5410u);
                    const uint32_t sg = prmt(db[2 * h], db[2 * h + 1], 0xF0B0u);
                    const uint32_t v = xp(mg | (sg & 0x80008000u));
                    const uint32_t ors = __reduce_or_sync(kFull, mg);
                    const uint32_t L0 = 32u - (uint32_t)__clz((int)(ors & 0x7FFFu));
                    const uint32_t L1 = 32u - (uint32_t)__clz((int)(ors >> 16));
                    const uint32_t n0 = L0 ? L0 + 1u : 0u, n1 = L1 ? L1 + 1u : 0u;
                    const uint32_t wp2 = ((uint32_t)lane + 1u) & 15u;
                    const bool hi = lane >= 16;
                    if (wp2 < (hi ? n1 : n0)) slots_w[wsum + (hi ? n0 : 0u) + wp2] = v;
                    wsum += n0 + n1;
                    lword |= (L0 | (L1 << 8)) << (16 * h);
                }
            } else {
#pragma unroll
                for (int u = 0; u < 4; ++u) {
                    const uint32_t m = __reduce_or_sync(kFull, ab[u]) & 0x7FFFFFu;
                    const uint32_t L = 32u - (uint32_t)__clz((int)m);
                    if (L) {   // uniform over the warp
                        const uint32_t v = xp(ab[u] | (db[u] & 0x80000000u));
                        if (widx <= L) slots_w[wsum + widx] = v;
                        wsum += L + 1;
                    }
                    lword |= L << (8 * u);
                }
            }
        } else {
#pragma unroll
            for (int u = 0; u < 4; ++u) {
                const float t = __fmul_rn(src.cur(g, u), r), tp = __fmul_rn(src.prev(g, u), r);
                tm = fmaxf(tm, fabsf(t));
                const int32_t q = __float2int_rn(t), qp = __float2int_rn(tp);
                const int32_t dd = q - qp;
                const uint32_t ab = (uint32_t)(dd < 0 ? -dd : dd);
                const uint32_t m = __reduce_or_sync(kFull, ab);
                const uint32_t L = 32u - (uint32_t)__clz((int)m);
                const uint32_t sg = __ballot_sync(kFull, dd < 0);
                if (L) {
                    uint32_t* slot = slots_w + wsum;
                    slot[0] = sg;   // every lane stores the same warp-uniform word
                    for (uint32_t k = 0; k < L; ++k) slot[k + 1] = __ballot_sync(kFull, ab & (1u << k));
                    wsum += L + 1;
                }
                lword |= L << (8 * u);
            }
        }
        if (lane == g) my_lw = lword;
    }
    guard = acc;
    tmax = tm;
    return wsum;
}

// The tile's outlier: the quantised code of its first element (thread 0 only needs it).
template <bool FAST>
__device__ __forceinline__ int32_t first_code(float x0, float r)
{
    const float t = __fmul_rn(x0, r);
    if (FAST) return (int32_t)(__float_as_uint(__fadd_rn(t, kRoundMagic)) - kRoundMagicBits);
    return __float2int_rn(t);
}

// Placement split in two.  Everything about a pending tile that is the same for all threads (scan of the sizes,
// layout of the warps' regions, capacity check, index entry, outlier, header, stream length) is done once, by warp 0,
// which leaves the result here; after a barrier each warp only copies its own region.
struct PlanShared {
    uint32_t* blob_out;       // where the pending tile's blob starts in the stream (nullptr: do not copy)
    uint32_t wbase[kWarps];   // each warp's first word inside the blob
    uint32_t padw;            // code-length words of the blob
    // what warp 0 worked out ahead of the barrier (laid_out != 0) and picks up again after it
    uint32_t laid_out, total, nT, lo, base;
};
// Hand-off of the scan's sizes from warps 2..7 to warp 0 (warp 1 requests the next tile's input meanwhile).
constexpr int kScanFirstWarp = 2, kScanWarps = kWarps - kScanFirstWarp;
struct ScanShared {
    uint32_t part[kWarps];    // sum of the sizes warp w fetched
    uint32_t ok[kWarps];      // 1 if every state that warp saw was published
    alignas(8) unsigned long long scanbar;   // the scanning warps arrive once their shares are written
};

struct EncodeShared {
    alignas(16) float xbuf[kTile + 8];                             // staged input tile (+ guard word in front)
    alignas(16) uint32_t slots[2][kBlocksPerTile * kSlotWords];    // encoded tiles: current and awaiting placement
    uint32_t warp_words[2][kWarps];
    PlanShared plan[2];                                            // placements alternate between the two cells
    ScanShared scan;
    uint32_t next_ticket;                                          // number of the tile after the current one
    alignas(8) unsigned long long bar;
};

// COMPACT: the kernel instance for launches whose tiles all fit the device at once, one tile per CTA: nothing is
// double buffered, which leaves room for one more CTA per SM.
template <bool COMPACT>
struct FusedSharedT {
    alignas(16) uint32_t blob[COMPACT ? 1 : 2][kBlobStageWords];     // staged blobs: current tile and the next one
    alignas(16) float ybuf[kWarps][(kBlocksPerWarp + 1) * kBlock];   // deltas, then sums (row 0 of a warp = guard)
    alignas(16) uint2 tbl[kBlocksPerTile];
    alignas(16) uint32_t slots[COMPACT ? 1 : 2][kBlocksPerTile * kSlotWords];
    BlobSpan span[2];
    float warp_total[kWarps];
    int32_t warp_total_i[kWarps];
    int32_t warp_total_i2[kWarps];
    uint32_t warp_words[2][kWarps];
    PlanShared plan[2];                                              // placements alternate between the two cells
    ScanShared scan;
    alignas(8) unsigned long long bar[2];
};
using FusedShared = FusedSharedT<false>;
using FusedSharedCompact = FusedSharedT<true>;

// A raw-mode tile can be staged by a bulk copy when it is full and starts on a 16-byte boundary.
__device__ __forceinline__ bool stageable_raw(const Job& job, uint32_t tile)
{
    const unsigned long long start = (unsigned long long)tile * kTile;
    return job.n - start >= (unsigned long long)kTile && (((uintptr_t)(job.x + start)) & 15u) == 0;
}


// An encoded tile sitting in shared memory until its place in the stream is known.  Placement is deferred by one
// tile: while a CTA encodes its next tile the sizes of the earlier tiles of all CTAs get published, so the scan of
// the deferred tile finds them without waiting.
struct Pending {
    bool valid;
    int job;
    uint32_t ticket;
    uint32_t buf;        // which half of the slots (and of the warps' sizes) holds it
    uint32_t wsum;       // this warp's payload words
    uint32_t my_lw;      // lanes 0..3: this warp's code-length words
    int32_t q_first;     // outlier (thread 0)
};

// What a CTA remembers about the last tile it placed: the anchor of its next scan.
struct Anchor {
    int job;             // -1: none yet
    uint32_t ticket;
    uint32_t incl;       // inclusive prefix (words) of that tile within its job
};

// Sum of the sizes of tiles [lo, hi) of the launch, by one warp: all states are fetched in one round trip.
__device__ __forceinline__ uint32_t sum_sizes_warp(const Workspace& ws, uint32_t lo, uint32_t hi, uint32_t epoch, int lane,
                                                   uint32_t& skip, uint32_t& status)
{
    skip = 0;
    if (hi <= lo) return 0;
    int budget = kSpinLimit >> 4;
    for (;;) {
        uint32_t sum = 0;
        bool good = true;
        for (uint32_t base = lo; base < hi; base += 256) {
            unsigned long long st[8];
#pragma unroll
            for (int k = 0; k < 8; ++k) {
                const uint32_t at = base + 32u * k + lane;
                st[k] = (at < hi) ? ld_state(ws.tile_state + at) : pack_state(epoch, 0u, 0u);
            }
#pragma unroll
            for (int k = 0; k < 8; ++k) {
                if ((uint32_t)(st[k] >> 33) == epoch) sum += (uint32_t)st[k];
                else good = false;
            }
        }
        sum = __reduce_add_sync(kFull, sum);
        if (__all_sync(kFull, good)) return sum;
        if (--budget == 0) { skip = 1; status |= kStTimeout; return 0; }
        __nanosleep(64);
    }
}


// First tile of the scan that places a tile of job `job_index`, given the tile this CTA placed last.
__device__ __forceinline__ uint32_t scan_begin(const Anchor& a, int job_index, const JobBatch& jb)
{
    return a.job == job_index ? a.ticket + 1 : jb.job[job_index].tile_begin;
}

// Warps 2..7, while warp 0 publishes and lays out: each fetches its share of the sizes of tiles [lo, hi) (window k
// of 32 tiles belongs to warp 2 + k mod 6, all loads of a warp in flight together), leaves the sum for warp 0 and
// arrives on the hand-off barrier.  One round trip to L2 for the whole scan.
__device__ __forceinline__ void scan_share(ScanShared& plan, const Workspace& ws, uint32_t lo, uint32_t hi, uint32_t epoch,
                                           int warp, int lane)
{
    uint32_t sum = 0;
    bool good = true;
    if (hi > lo) {
        const uint32_t nwin = (hi - lo + 31u) >> 5;
#pragma unroll 4
        for (uint32_t w = (uint32_t)(warp - kScanFirstWarp); w < nwin; w += kScanWarps) {
            const uint32_t at = lo + 32u * w + (uint32_t)lane;
            if (at < hi) {
                const unsigned long long st = ld_state(ws.tile_state + at);
                if ((uint32_t)(st >> 33) == epoch) sum += (uint32_t)st;
                else good = false;
            }
        }
    }
    sum = __reduce_add_sync(kFull, sum);
    good = __all_sync(kFull, good);
    if (lane == 0) {
        plan.part[warp] = sum;
        plan.ok[warp] = good ? 1u : 0u;
        mbar_arrive(&plan.scanbar);
    }
}

// What warp 0 keeps of a plan for the stores it does once the other warps have been released.
struct Planned {
    uint32_t* blob_out;
    uint32_t incl;
    bool go;
};

// Warp 0, any time after the pending tile was encoded (the encoder does it while it waits for the next input
// tile): everything about its placement that does not depend on the other CTAs' sizes.
__device__ __forceinline__ void lay_out_pending(PlanShared& plan, const Pending& c, const uint32_t* pend_words, const Anchor& anchor,
                                                const JobBatch& jb, int lane)
{
    const Job& job = jb.job[c.job];
    const uint32_t tile = c.ticket - job.tile_begin;
    const unsigned long long start = (unsigned long long)tile * kTile;
    const uint32_t nT = (uint32_t)((job.n + kTile - 1) / kTile);
    const uint32_t len = (uint32_t)((job.n - start < (unsigned long long)kTile) ? (job.n - start) : kTile);
    const uint32_t padw = (((len + kBlock - 1) / kBlock) + 3) >> 2;
    // exclusive scan of the warps' sizes across lanes 0..7
    const uint32_t ww = lane < kWarps ? pend_words[lane] : 0u;
    uint32_t inc = ww;
#pragma unroll
    for (int k = 1; k < kWarps; k <<= 1) {
        const uint32_t up = __shfl_up_sync(kFull, inc, k);
        if (lane >= k) inc += up;
    }
    const uint32_t total = 1 + padw + __shfl_sync(kFull, inc, kWarps - 1);
    if (lane < kWarps) plan.wbase[lane] = 1 + padw + inc - ww;
    if (lane == 0) {
        plan.padw = padw;
        plan.total = total; plan.nT = nT;
        plan.lo = scan_begin(anchor, c.job, jb);
        plan.base = anchor.job == c.job ? anchor.incl : 0u;
        plan.laid_out = 1u;
    }
    __syncwarp();
}

// Warp 0, after the barrier that follows a tile's encoding pass: publishes the size of the tile just encoded
// (`ticket`, sizes in `cur_words`) and completes the plan of the pending one: the scan's sum from the other warps'
// shares (`shared_scan`; a blocking scan of its own when a size was not published yet, or when there are no
// shares), capacity check, target address.
__device__ __forceinline__ Planned announce_and_plan(PlanShared& plan, ScanShared& scan, const uint32_t* cur_words, uint32_t cur_padw,
                                                     uint32_t ticket, bool have_cur, const Pending& c, const uint32_t* pend_words,
                                                     Anchor& anchor, bool shared_scan, uint32_t scan_parity, const JobBatch& jb,
                                                     const Workspace& ws, uint32_t epoch, int lane, uint32_t& status)
{
    Planned d;
    d.blob_out = nullptr; d.incl = 0; d.go = false;
    if (have_cur) {
        const uint32_t ww = lane < kWarps ? cur_words[lane] : 0u;
        const uint32_t total = 1 + cur_padw + __reduce_add_sync(kFull, ww);
        if (lane == 0 && ticket != ws.skip_publish) st_state(ws.tile_state + ticket, pack_state(epoch, 0u, total));
    }
    if (!c.valid) return d;
    if (!plan.laid_out) lay_out_pending(plan, c, pend_words, anchor, jb, lane);
    const uint32_t total = plan.total, nT = plan.nT, lo = plan.lo, base = plan.base;
    const Job& job = jb.job[c.job];
    uint32_t skip = 0, between = 0;
    bool have = false;
    if (shared_scan) {
        if (!mbar_wait(&scan.scanbar, scan_parity)) status |= kStTimeout;
        const uint32_t ps = (lane >= kScanFirstWarp && lane < kWarps) ? scan.part[lane] : 0u;
        const uint32_t ok = (lane >= kScanFirstWarp && lane < kWarps) ? scan.ok[lane] : 1u;
        between = __reduce_add_sync(kFull, ps);
        have = __all_sync(kFull, ok != 0u);
    }
    if (!have) between = sum_sizes_warp(ws, lo, c.ticket, epoch, lane, skip, status);
    const uint32_t excl = base + between;
    anchor.incl = excl + total;
    d.incl = excl + total;
    const unsigned long long blob_word0 = (unsigned long long)kHeaderWords + nT + excl;
    const bool fits = (blob_word0 + total) * 4ull <= job.out_cap;
    if (!fits) status |= kStCapacity;
    d.go = fits && !skip;
    d.blob_out = job.out + blob_word0;
    __syncwarp();
    if (lane == 0) {
        plan.blob_out = d.go ? d.blob_out : nullptr;
        plan.laid_out = 0u;   // the next tile planned in this cell starts afresh
    }
    return d;
}

// Warp 0, once the other warps are copying: outlier, index entry, stream length, header of the tile just planned.
__device__ __forceinline__ void finish_plan(const Planned& d, const Pending& c, const JobBatch& jb, float eb_abs, float s, int lane)
{
    const Job& job = jb.job[c.job];
    const uint32_t tile = c.ticket - job.tile_begin;
    const uint32_t nT = (uint32_t)((job.n + kTile - 1) / kTile);
    if (lane == 0) {
        if (d.go) {
            d.blob_out[0] = (uint32_t)c.q_first;
            job.out[kHeaderWords + tile] = d.incl;
        }
        if (tile == nT - 1) *job.out_bytes = (size_t)(((unsigned long long)kHeaderWords + nT + d.incl) * 4ull);
    }
    if (tile == 0) write_header(job.out, lane, job.n, eb_abs, s, nT);
}

// Every warp, after the barrier that follows the plan: copy its own region of the pending tile.
__device__ __forceinline__ void copy_planned(const PlanShared& plan, const Pending& c, const uint32_t* __restrict__ slots_w,
                                             int warp, int lane)
{
    uint32_t* __restrict__ blob_out = plan.blob_out;
    if (blob_out == nullptr) return;
    uint32_t* __restrict__ dst = blob_out + plan.wbase[warp];
    for (uint32_t i = lane; i < c.wsum; i += 32) dst[i] = slots_w[i];
    if (lane < 4 && (uint32_t)(4 * warp + lane) < plan.padw) blob_out[1 + 4 * warp + lane] = c.my_lw;
}

// First half of the placement of a pending tile, by the whole CTA, after the barrier that made the current tile's
// sizes visible (have_cur) or at the end of the launch: warps 2..7 fetch the scan's sizes while warp 0 publishes
// and lays out, then warp 0 completes the plan.  The caller follows with a barrier, copy_planned by every warp and
// finish_plan by warp 0.  Uniform over the CTA.
__device__ __forceinline__ Planned plan_pending(PlanShared& plan, ScanShared& scan, const uint32_t* cur_words, uint32_t cur_padw,
                                                uint32_t ticket, bool have_cur, const Pending& c, const uint32_t* pend_words,
                                                Anchor& anchor, uint32_t& scan_parity, const JobBatch& jb, const Workspace& ws,
                                                uint32_t epoch, int warp, int lane, uint32_t& status)
{
    Planned pl;
    pl.blob_out = nullptr; pl.incl = 0; pl.go = false;
    if (warp == 0) {
        pl = announce_and_plan(plan, scan, cur_words, cur_padw, ticket, have_cur, c, pend_words, anchor, c.valid, scan_parity, jb, ws,
                               epoch, lane, status);
    } else if (c.valid && warp >= kScanFirstWarp) {
        scan_share(scan, ws, scan_begin(anchor, c.job, jb), c.ticket, epoch, warp, lane);
    }
    if (c.valid) {
        scan_parity ^= 1u;
        anchor.job = c.job; anchor.ticket = c.ticket;   // every warp tracks which tile was placed last; warp 0 also its prefix
    }
    return pl;
}

// ------------------------------------------------------------------------------------------------ compress

__global__ void __launch_bounds__(kThreads, 4) encode_raw_kernel(JobBatch jb, Workspace ws, Params hp, int use_dev_params)
{
    pdl_enter();
    extern __shared__ __align__(16) unsigned char smem_raw[];
    EncodeShared& sh = *reinterpret_cast<EncodeShared*>(smem_raw);
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const uint32_t epoch = *reinterpret_cast<volatile uint32_t*>(ws.epoch);
    uint32_t status = 0;
    Params prm = hp;
    if (use_dev_params) prm = *ws.params;
    const float r = prm.r, s = prm.s, eb_abs = prm.eb_abs;
    float* const xt = &sh.xbuf[4];

    // thread 0 starts the bulk copy of tile `t` into the staging buffer when that tile can be staged
    auto stage = [&](uint32_t t) {
        if (t < jb.total_tiles && prm.valid) {
            const Job& jn = jb.job[find_job(jb, t)];
            const uint32_t tn = t - jn.tile_begin;
            if (jn.n && stageable_raw(jn, tn)) {
                mbar_expect_tx(&sh.bar, kTile * 4);
                bulk_load(xt, jn.x + (unsigned long long)tn * kTile, kTile * 4, &sh.bar);
            }
        }
    };
    // Tiles are handed out in order by a device-wide counter, one tile ahead of the encoding (the thread that
    // requests a tile's input takes its number): a CTA that gets fewer issue slots than its neighbours simply takes
    // fewer tiles, and every tile before a given one was taken earlier than it.
    auto take_next = [&]() {
        const uint32_t t = atomicAdd(ws.ticket, 1u);
        sh.next_ticket = t;
        stage(t);
    };
    if (tid == 0) {
        mbar_init(&sh.bar, 1);
        mbar_init(&sh.scan.scanbar, kScanWarps);
        sh.plan[0].laid_out = 0u; sh.plan[1].laid_out = 0u;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
        take_next();
    }
    __syncthreads();
    uint32_t scan_par = 0;   // phase parity of the scan's hand-off barrier
    uint32_t fills = 0;    // completed bulk copies (phase parity of the mbarrier)
    uint32_t p = 0;        // half of the slots the current tile is encoded into
    Pending pend;
    pend.valid = false;
    Anchor anchor;
    anchor.job = -1; anchor.ticket = 0; anchor.incl = 0;
    const Xpose xp(lane);

    for (;;) {
        const uint32_t ticket = sh.next_ticket;   // written before the last barrier
        if (ticket >= jb.total_tiles) break;
        const int j = find_job(jb, ticket);
        const Job& job = jb.job[j];
        const uint32_t tile = ticket - job.tile_begin;
        const unsigned long long n = job.n;
        const bool staged = prm.valid && n && stageable_raw(job, tile);

        if (n == 0 || !prm.valid) {   // a job without elements still owns one tile number: header and length only
            const bool hdr = prm.valid && job.out_cap >= (unsigned)kHeaderBytes;
            __syncthreads();   // every thread has read this tile's number
            if (tid == 0) {
                st_state(ws.tile_state + ticket, pack_state(epoch, 0u, 0u));
                if (tile == 0) *job.out_bytes = hdr ? kHeaderBytes : 0;
                take_next();   // nothing was staged for this tile, and the buffer's last readers are past a barrier
            }
            if (hdr && tile == 0) write_header(job.out, tid, 0, eb_abs, s, 0);
            __syncthreads();   // the next tile's number is visible
            continue;
        }

        const unsigned long long start = (unsigned long long)tile * kTile;
        const uint32_t len = (uint32_t)((n - start < (unsigned long long)kTile) ? (n - start) : kTile);
        const uint32_t nb = (len + kBlock - 1) / kBlock;

        // ---- single pass over the warp's blocks: quantise, delta, code length, planes -> this warp's region
        uint32_t* slots_w = sh.slots[p] + kSlotWords * kBlocksPerWarp * warp;
        uint32_t my_lw = 0, wsum = 0;
        int32_t q_first = 0;
        float guard = 0.0f, tmax = 0.0f;
        bool need_int = !staged;
        // while the input tile is on its way, warp 0 lays out the pending tile (its cell of the plan is free: the
        // placement before it used the other one)
        if (warp == 0 && pend.valid) lay_out_pending(sh.plan[scan_par], pend, sh.warp_words[pend.buf], anchor, jb, lane);
        if (staged) {
            const bool landed = mbar_wait(&sh.bar, fills & 1u);
            ++fills;
            if (!landed) status |= kStTimeout;   // carry on with whatever is staged: the result is flagged invalid
            if (tid == 0) xt[-1] = xt[0];        // the tile's first element is its own predecessor
            const SrcStaged src{xt + 512 * warp + lane};
            wsum = encode_blocks<true>(src, r, slots_w, lane, xp, my_lw, guard, tmax);
            q_first = first_code<true>(src.cur(0, 0), r);
            need_int = __any_sync(kFull, !(guard < kGuardExact));
            if (!need_int && __any_sync(kFull, guard >= kGuardSmall)) {   // codes beyond 2^15 raise the warning
                float tm = 0.0f;
#pragma unroll 1
                for (int g = 0; g < 4; ++g)
#pragma unroll
                    for (int u = 0; u < 4; ++u) tm = fmaxf(tm, fabsf(__fmul_rn(src.cur(g, u), r)));
                if (tm > 32768.5f) status |= kStPrecision;
            }
        }
        if (need_int) {
            const SrcGlobal src{job.x + start, (uint32_t)(512 * warp + lane), len - 1};
            wsum = encode_blocks<false>(src, r, slots_w, lane, xp, my_lw, guard, tmax);
            q_first = first_code<false>(src.cur(0, 0), r);
            if (!(tmax < 1073741824.0f)) status |= kStRange;
            else if (tmax > 32768.5f) status |= kStPrecision;
        }
        if (lane == 0) sh.warp_words[p][warp] = wsum;
        __syncthreads();   // sizes of all warps are visible; the staged tile has been consumed
        PlanShared& cell = sh.plan[scan_par];
        const Planned pl = plan_pending(cell, sh.scan, sh.warp_words[p], (nb + 3) >> 2, ticket, true, pend, sh.warp_words[pend.buf],
                                        anchor, scan_par, jb, ws, epoch, warp, lane, status);
        if (tid == 32) take_next();   // by warp 1, while warp 0 completes the plan
        __syncthreads();   // the plan and the next tile's number are visible
        if (pend.valid) {
            copy_planned(cell, pend, sh.slots[pend.buf] + kSlotWords * kBlocksPerWarp * warp, warp, lane);
            if (warp == 0) finish_plan(pl, pend, jb, eb_abs, s, lane);
        }
        pend.valid = true; pend.job = j; pend.ticket = ticket; pend.buf = p; pend.wsum = wsum; pend.my_lw = my_lw;
        pend.q_first = q_first;
        p ^= 1u;
    }
    if (pend.valid) {
        __syncthreads();
        PlanShared& cell = sh.plan[scan_par];
        const Planned pl = plan_pending(cell, sh.scan, nullptr, 0, 0, false, pend, sh.warp_words[pend.buf], anchor, scan_par, jb, ws,
                                        epoch, warp, lane, status);
        __syncthreads();
        copy_planned(cell, pend, sh.slots[pend.buf] + kSlotWords * kBlocksPerWarp * warp, warp, lane);
        if (warp == 0) finish_plan(pl, pend, jb, eb_abs, s, lane);
    }

    // never leave with a bulk copy in flight into this CTA's shared memory: every copy that was started has been
    // waited for by the iteration that consumed it, except after an expired wait; then give it one more bounded wait
    if (tid == 0 && (status & kStTimeout)) (void)mbar_wait(&sh.bar, (fills + 1u) & 1u);
    if (status) atomicOr(ws.status, status);
    finish_launch(ws, epoch, tid, ws.ticket);
}

// ------------------------------------------------------------------------------------------------ fused hop

// out = compress(decompress(in_c) + local) per tile, with no uncompressed intermediate in global memory.
template <bool COMPACT>
__global__ void __launch_bounds__(kThreads, COMPACT ? 4 : 3) encode_fused_kernel(JobBatch jb, Workspace ws)
{
    pdl_enter();
    extern __shared__ __align__(16) unsigned char smem_raw[];
    using Shared = FusedSharedT<COMPACT>;
    Shared& sh = *reinterpret_cast<Shared*>(smem_raw);
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const uint32_t epoch = *reinterpret_cast<volatile uint32_t*>(ws.epoch);
    const uint32_t G = gridDim.x;
    uint32_t status = 0;
    uint32_t fills0 = 0, fills1 = 0;   // bulk copies completed per staging buffer
    uint32_t p = 0;                    // half of the slots and staging buffer of the current tile
    float pend_eb = 0.0f, pend_s = 1.0f;   // bound and step of the pending tile's job (header fields)
    Pending pend;
    pend.valid = false;
    Anchor anchor;
    anchor.job = -1; anchor.ticket = 0; anchor.incl = 0;
    const Xpose xp(lane);
    int cur_job = -1;
    StreamInfo h1, h2;
    h1.ok = h2.ok = false; h1.n = h2.n = 0; h1.nT = h2.nT = 0; h1.s = h2.s = 1.0f; h1.eb_abs = h2.eb_abs = 0.0f;
    bool job_ok = false;
    float r = 1.0f;   // reciprocal of the current job's step

    // The first thread of warp 1 requests the blobs: it does so while warp 0 plans a placement, when the other
    // warps have nothing to do.
    StagePipe pipe;   // thread 32 only
    if (tid == 0) {
        mbar_init(&sh.bar[0], 1);
        mbar_init(&sh.bar[1], 1);
        mbar_init(&sh.scan.scanbar, kScanWarps);
        sh.plan[0].laid_out = 0u; sh.plan[1].laid_out = 0u;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    __syncthreads();
    uint32_t scan_par = 0;   // phase parity of the scan's hand-off barrier
    if (tid == 32) {
        pipe.fetch(jb, blockIdx.x, cur_job, h1);
        pipe.stage(sh, jb, blockIdx.x, cur_job, h1, 0);
        if (!COMPACT) pipe.fetch(jb, blockIdx.x + G, cur_job, h1);
    }
    __syncthreads();
    // requests the next tile's blob into the other staging buffer (its readers finished before the last barrier), then
    // fetches the index entries of the tile after it; a barrier follows before the span is read
    auto stage_next = [&](uint32_t ticket) {
        if (!COMPACT && tid == 32) {   // a compact launch has one tile per CTA: nothing comes next
            pipe.stage(sh, jb, ticket + G, cur_job, h1, p ^ 1u);
            pipe.fetch(jb, ticket + 2 * G, cur_job, h1);
        }
    };

    for (uint32_t ticket = blockIdx.x; ticket < jb.total_tiles; ticket += G, p ^= (COMPACT ? 0u : 1u)) {
        const int j = find_job(jb, ticket);
        const Job& job = jb.job[j];
        const uint32_t tile = ticket - job.tile_begin;
        const unsigned long long n = job.n;
        const uint32_t nT = (uint32_t)((n + kTile - 1) / kTile);
        if (j != cur_job) {
            cur_job = j;
            h1 = read_header(job.in_c, job.in_cap);
            job_ok = h1.ok && h1.n == n;
            if (job.in_c2) {
                h2 = read_header(job.in_c2, job.in2_cap);
                job_ok = job_ok && h2.ok && h2.n == n && __float_as_uint(h2.s) == __float_as_uint(h1.s);
            }
            r = __fdiv_rn(1.0f, h1.s);
        }
        const float s = h1.s, eb_abs = h1.eb_abs;

        const BlobSpan sp = sh.span[p];
        if (sp.staged) {   // a copy was requested for this tile: always consume it, whatever happens next
            const uint32_t fl = p ? fills1 : fills0;
            if (!mbar_wait(&sh.bar[p], fl & 1u)) status |= kStTimeout;
            if (p) ++fills1; else ++fills0;
        }

        if (!job_ok || n == 0) {
            if (!job_ok) status |= kStBadStream;
            const bool hdr = job_ok && job.out_cap >= (unsigned)kHeaderBytes;
            if (tid == 0) {
                st_state(ws.tile_state + ticket, pack_state(epoch, 0u, 0u));
                if (tile == 0) *job.out_bytes = hdr ? kHeaderBytes : 0;
            }
            if (hdr && tile == 0) write_header(job.out, tid, 0, eb_abs, s, 0);
            stage_next(ticket);
            __syncthreads();
            continue;
        }

        const unsigned long long start = (unsigned long long)tile * kTile;
        const uint32_t len = (uint32_t)((n - start < (unsigned long long)kTile) ? (n - start) : kTile);
        const uint32_t nb = (len + kBlock - 1) / kBlock;
        const uint32_t padw = (nb + 3) >> 2;
        const uint32_t last = len - 1;
        float* yrows = sh.ybuf[warp];
        const float* __restrict__ loc = job.x ? job.x + start : nullptr;
        float* __restrict__ yout = job.y ? job.y + start : nullptr;
        const bool deq = (job.flags & 1u) != 0;
        // reduce operation (bits 1..2 of the flags): 0 = sum, 1 = max, 2 = min, 3 = average (a sum on every hop);
        // of two operands that compare equal Max and Min keep the decoded one
        const uint32_t op = (job.flags >> 1) & 3u;
        const bool summing = op == 0u || op == 3u;
        auto combine = [&](float a, float b) {
            return op == 1u ? ((a < b) ? b : a) : op == 2u ? ((b < a) ? b : a) : __fadd_rn(a, b);
        };

        // ---- front end: decode + add, leaving the sums in this warp's rows of ybuf (swizzled), row 0 = guard
        int mode = 2;   // 1: fp32 front end from the staged blob, 2: integer front end from global memory
        bool bad_tile = false;
        if (sp.staged) {
            // this thread's 16 consecutive elements of the local operand are needed after the scan: pull their lines
            // towards L2 now, load them (128-bit when aligned) when they are used
            const float* lp = loc + 512 * warp + 16 * lane;
            const unsigned long long blob0 = (unsigned long long)kHeaderWords + h1.nT;
            const uint32_t shift = (uint32_t)(((uintptr_t)(job.in_c + blob0 + sp.w_beg) & 15u) >> 2);
            const uint32_t* sb = sh.blob[p] + shift;
            mode = describe_staged(sh.tbl, sb, sp.w_end - sp.w_beg, lane, warp);
            if (mode == 0) bad_tile = true;
            if (mode == 1) {
                decode_blocks_f32<(COMPACT ? 1 : 4)>(sh.tbl + kBlocksPerWarp * warp, yrows + 32, lane, xp);
                __syncwarp();
                // lane 0 needs the local operand's element before the warp's first one after the barrier below
                const float lprev = (lane == 0 && warp != 0) ? __ldg(loc + 512 * warp - 1) : 0.0f;
                float v[16];
                float before;
                const float total = decode_scan_f32(yrows + 32, lane, v, before);
                if (lane == 0) sh.warp_total[warp] = total;
                const float outlier = (float)(int32_t)sb[0];
                __syncthreads();   // warp totals
                float base = outlier;
                for (int w = 0; w < warp; ++w) base = __fadd_rn(base, sh.warp_total[w]);
                // the element before this warp's first one is the last element of the previous warp: its code is `base`
                if (lane == 0) {
                    float yprev;
                    if (warp == 0) yprev = combine(__fmul_rn(__fadd_rn(v[0], base), s), __ldg(loc));
                    else yprev = combine(__fmul_rn(base, s), lprev);
                    yrows[31 ^ 12] = yprev;   // guard row, element 31 under the swizzle of the row before row 0
                }
                base = __fadd_rn(base, before);   // integers below 2^24: any order of addition is exact
                const int sw = (lane >> 1) & 3;
                float4* row = reinterpret_cast<float4*>(yrows + 32 + 16 * lane);
                float4* gout = yout ? reinterpret_cast<float4*>(yout + 512 * warp + 16 * lane) : nullptr;
                // alignment and the presence of an uncompressed output are the same for every thread of the launch's job
                const bool lvec = (((uintptr_t)loc) & 15u) == 0;
                const bool store = gout != nullptr && !deq;
                const bool gvec = (((uintptr_t)yout) & 15u) == 0;
                if (summing && lvec && (!store || gvec)) {
                    // Global accesses are made warp-contiguous (access c of the warp covers 512 consecutive bytes)
                    // and the 16 consecutive elements a thread works on are exchanged through the warp's rows, whose
                    // deltas the scan has consumed: a 128-bit access with the lanes 64 bytes apart is replayed.
                    float4* row_w = reinterpret_cast<float4*>(yrows + 32);
                    const float4* lw = reinterpret_cast<const float4*>(loc + 512 * warp);
#pragma unroll
                    for (int c = 0; c < 4; ++c) {
                        const int f = 32 * c + lane, t = f >> 2;
                        row_w[4 * t + ((f & 3) ^ ((t >> 1) & 3))] = __ldg(lw + f);
                    }
                    __syncwarp();
                    float4 l[4];
#pragma unroll
                    for (int c = 0; c < 4; ++c) l[c] = row[c ^ sw];
#pragma unroll
                    for (int c = 0; c < 4; ++c) {
                        float4 o;
                        o.x = __fadd_rn(__fmul_rn(__fadd_rn(v[4 * c + 0], base), s), l[c].x);
                        o.y = __fadd_rn(__fmul_rn(__fadd_rn(v[4 * c + 1], base), s), l[c].y);
                        o.z = __fadd_rn(__fmul_rn(__fadd_rn(v[4 * c + 2], base), s), l[c].z);
                        o.w = __fadd_rn(__fmul_rn(__fadd_rn(v[4 * c + 3], base), s), l[c].w);
                        row[c ^ sw] = o;
                    }
                    if (store) {
                        __syncwarp();
                        float4* gw = reinterpret_cast<float4*>(yout + 512 * warp);
#pragma unroll
                        for (int c = 0; c < 4; ++c) {
                            const int f = 32 * c + lane, t = f >> 2;
                            gw[f] = row_w[4 * t + ((f & 3) ^ ((t >> 1) & 3))];
                        }
                    }
                } else {
#pragma unroll
                    for (int c = 0; c < 4; ++c) {
                        float4 l, o;
                        l.x = __ldg(lp + 4 * c); l.y = __ldg(lp + 4 * c + 1); l.z = __ldg(lp + 4 * c + 2); l.w = __ldg(lp + 4 * c + 3);
                        o.x = combine(__fmul_rn(__fadd_rn(v[4 * c + 0], base), s), l.x);
                        o.y = combine(__fmul_rn(__fadd_rn(v[4 * c + 1], base), s), l.y);
                        o.z = combine(__fmul_rn(__fadd_rn(v[4 * c + 2], base), s), l.z);
                        o.w = combine(__fmul_rn(__fadd_rn(v[4 * c + 3], base), s), l.w);
                        row[c ^ sw] = o;
                        if (store) { float* g = reinterpret_cast<float*>(gout + c); g[0] = o.x; g[1] = o.y; g[2] = o.z; g[3] = o.w; }
                    }
                }
                __syncwarp();
            }
        }
        if (!bad_tile && mode == 2) {
            // integer front end, one element per lane; ragged tails repeat the last element
            const TileDesc d1 = describe_tile(job.in_c, job.in_cap, h1, tile, lane);
            TileDesc d2 = d1;
            if (job.in_c2) d2 = describe_tile(job.in_c2, job.in2_cap, h2, tile, lane);
            if (!d1.ok || !d2.ok) bad_tile = true;
            else {
                int32_t qa[kBlocksPerWarp], qb[kBlocksPerWarp];
                decode_blocks_int(d1, warp, lane, qa);
                if (job.in_c2) decode_blocks_int(d2, warp, lane, qb);
                if (lane == 31) {
                    sh.warp_total_i[warp] = qa[kBlocksPerWarp - 1];
                    if (job.in_c2) sh.warp_total_i2[warp] = qb[kBlocksPerWarp - 1];
                }
                __syncthreads();   // warp totals
                int32_t base_a = d1.outlier, base_b = d2.outlier;
                for (int w = 0; w < warp; ++w) {
                    base_a += sh.warp_total_i[w];
                    if (job.in_c2) base_b += sh.warp_total_i2[w];
                }
                const uint32_t e0 = (uint32_t)(512 * warp + lane);
#pragma unroll
                for (int i = 0; i < kBlocksPerWarp; ++i) {
                    uint32_t e = e0 + 32u * i;
                    const bool inside = e <= last;
                    if (!inside) e = last;
                    const float xa = __fmul_rn(__int2float_rn(base_a + qa[i]), s);
                    const float xb = job.in_c2 ? __fmul_rn(__int2float_rn(base_b + qb[i]), s) : __ldg(loc + e);
                    const float yv = combine(xa, xb);
                    yrows[32 * (i + 1) + (lane ^ ((i & 3) << 2))] = yv;
                    if (yout && !deq && inside) yout[e] = yv;
                }
                if (lane == 0) {
                    float yprev;
                    if (warp == 0) {
                        yprev = yrows[32];   // own first element (row 1, lane 0, swizzle 0)
                    } else {
                        const uint32_t ep = min((uint32_t)(512 * warp - 1), last);
                        const float xa = __fmul_rn(__int2float_rn(base_a), s);
                        const float xb = job.in_c2 ? __fmul_rn(__int2float_rn(base_b), s) : __ldg(loc + ep);
                        yprev = combine(xa, xb);
                    }
                    yrows[31 ^ 12] = yprev;
                }
                __syncwarp();
            }
        }
        if (bad_tile) {   // uniform: keep the scan consistent for the tiles that follow, write nothing
            status |= kStBadStream;
            if (tid == 0) {
                st_state(ws.tile_state + ticket, pack_state(epoch, 0u, 0u));
                if (tile == nT - 1) *job.out_bytes = 0;
            }
            stage_next(ticket);
            __syncthreads();
            continue;
        }

        // ---- back end: encode the sums
        uint32_t* slots_w = sh.slots[p] + kSlotWords * kBlocksPerWarp * warp;
        uint32_t my_lw = 0, wsum = 0;
        int32_t q_first = 0;
        float guard = 0.0f, tmax = 0.0f;
        const SrcSwizzled src(yrows, lane);
        wsum = encode_blocks<true, (COMPACT ? 1 : 4)>(src, r, slots_w, lane, xp, my_lw, guard, tmax);
        q_first = first_code<true>(src.cur(0, 0), r);
        const bool need_int = __any_sync(kFull, !(guard < kGuardExact));
        if (need_int) {
            wsum = encode_blocks<false, (COMPACT ? 1 : 4)>(src, r, slots_w, lane, xp, my_lw, guard, tmax);
            q_first = first_code<false>(src.cur(0, 0), r);
            if (!(tmax < 1073741824.0f)) status |= kStRange;
            else if (tmax > 32768.5f) status |= kStPrecision;
        } else if (__any_sync(kFull, guard >= kGuardSmall)) {
            float tm = 0.0f;
#pragma unroll 1
            for (int g = 0; g < 4; ++g)
#pragma unroll
                for (int u = 0; u < 4; ++u) tm = fmaxf(tm, fabsf(__fmul_rn(src.cur(g, u), r)));
            if (tm > 32768.5f) status |= kStPrecision;
        }
        if (yout && deq) {   // owner's copy as the dequantised value float(q(y)) * s
            const uint32_t e0 = (uint32_t)(512 * warp + lane);
#pragma unroll 1
            for (int g = 0; g < 4; ++g)
#pragma unroll
                for (int u = 0; u < 4; ++u) {
                    const uint32_t e = e0 + 32u * (4 * g + u);
                    if (e <= last) yout[e] = __fmul_rn(__int2float_rn(__float2int_rn(__fmul_rn(src.cur(g, u), r))), s);
                }
        }
        if (lane == 0) sh.warp_words[p][warp] = wsum;
        __syncthreads();   // sizes of all warps
        PlanShared& cell = sh.plan[scan_par];
        const Planned pl = plan_pending(cell, sh.scan, sh.warp_words[p], padw, ticket, true, pend, sh.warp_words[pend.buf], anchor,
                                        scan_par, jb, ws, epoch, warp, lane, status);
        stage_next(ticket);
        __syncthreads();   // the plan and the next tile's span are visible
        if (pend.valid) {
            copy_planned(cell, pend, sh.slots[pend.buf] + kSlotWords * kBlocksPerWarp * warp, warp, lane);
            if (warp == 0) finish_plan(pl, pend, jb, pend_eb, pend_s, lane);
        }
        pend.valid = true; pend.job = j; pend.ticket = ticket; pend.buf = p; pend.wsum = wsum; pend.my_lw = my_lw;
        pend.q_first = q_first;
        pend_eb = eb_abs; pend_s = s;
    }
    if (pend.valid) {
        __syncthreads();
        PlanShared& cell = sh.plan[scan_par];
        const Planned pl = plan_pending(cell, sh.scan, nullptr, 0, 0, false, pend, sh.warp_words[pend.buf], anchor, scan_par, jb, ws,
                                        epoch, warp, lane, status);
        __syncthreads();
        copy_planned(cell, pend, sh.slots[pend.buf] + kSlotWords * kBlocksPerWarp * warp, warp, lane);
        if (warp == 0) finish_plan(pl, pend, jb, pend_eb, pend_s, lane);
    }
    if (tid == 0 && (status & kStTimeout)) {
        (void)mbar_wait(&sh.bar[0], (fills0 + 1u) & 1u);
        (void)mbar_wait(&sh.bar[1], (fills1 + 1u) & 1u);
    }
    if (status) atomicOr(ws.status, status);
    finish_launch(ws, epoch, tid);
}

// ------------------------------------------------------------------------------------------------ blob copy

// One forwarding hop of compressed bytes whose length lives on the device (grid.y = job).
__global__ void __launch_bounds__(256) copy_kernel(CopyBatch cb, Workspace ws)
{
    pdl_enter();
    const CopyJob& job = cb.job[blockIdx.y];
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

// Every forwarding hop of an Allgather stage (grid.y = chain).  A thread carries its 16-byte pieces through all the
// hops: each hop loads the piece from where the previous hop stored it (the same thread's own store, so no
// synchronisation is needed) and stores it into the next rank's slot.
__global__ void __launch_bounds__(256) copy_chain_kernel(ChainBatch cb, Workspace ws)
{
    pdl_enter();
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
            take(a0.x, b0.x, 0); take(a0.y, b0.y, 1); take(a0.z, b0.z, 2); take(a0.w, b0.w, 3);
            take(a1.x, b1.x, 4); take(a1.y, b1.y, 5); take(a1.z, b1.z, 6); take(a1.w, b1.w, 7);
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

int g_raw_ctas_per_sm = 0, g_fused_ctas_per_sm = 0, g_decode_ctas_per_sm = 0, g_compact_ctas_per_sm = 0;
unsigned long long g_launches = 0;   // kernels launched by this library in this process

}  // namespace

// ------------------------------------------------------------------------------------------------ launchers

unsigned long long launch_count() { return g_launches; }

// Launch with programmatic stream serialisation (see pdl_enter); ZCCL_PDL=0 in the environment turns it off.
// EARLY = false keeps a kernel fully serialised behind its predecessor.  The fused hop needs that: its tiles are
// dealt round-robin over a grid that must be resident as a whole (a CTA's scan waits for tiles of other CTAs), and
// CTAs dispatched onto SMs that still run another kernel's CTAs do not all fit (the SM keeps that kernel's
// shared-memory configuration), which left part of the grid waiting behind the resident part.  The other kernels
// make no such assumption: tiles handed out by a counter, or CTAs that never wait for one another.
// ZCCL_COMPACT in the environment: 0 never use the compact instance of the fused kernel, 1 (default) use it for
// launches that exceed the persistent instance's resident CTAs but fit the compact one's, 2 use it whenever the
// tiles fit (measured: a little faster up to 128 tiles, slower at 256).
static bool lanes_engine()
{
    static const bool on = [] { const char* e = getenv("ZCCL_ENGINE"); return !(e && e[0] == '0'); }();
    return on;
}

static int compact_mode()
{
    static const int m = [] { const char* e = getenv("ZCCL_COMPACT"); return e ? atoi(e) : 1; }();
    return m;
}

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
    if (mode == kEncodeRaw && lanes_engine()) {
        g_launches += ws.slots ? 2 : 1;
        return launch_encode_lanes(jb, ws, device_params, host_params, sm_count, st);
    }
    if (mode == kEncodeFused && lanes_engine() && ws.slots) {
        g_launches += 2;
        return launch_hop_lanes(jb, ws, sm_count, st);
    }
    if (g_raw_ctas_per_sm == 0) {
        cudaError_t e = cudaFuncSetAttribute(encode_raw_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                             (int)sizeof(EncodeShared));
        if (e != cudaSuccess) return e;
        e = cudaFuncSetAttribute(encode_fused_kernel<false>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)sizeof(FusedShared));
        if (e != cudaSuccess) return e;
        e = cudaFuncSetAttribute(encode_fused_kernel<true>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)sizeof(FusedSharedCompact));
        if (e != cudaSuccess) return e;
        int a = 0, b = 0, c = 0;
        cudaOccupancyMaxActiveBlocksPerMultiprocessor(&a, encode_raw_kernel, kThreads, sizeof(EncodeShared));
        cudaOccupancyMaxActiveBlocksPerMultiprocessor(&b, encode_fused_kernel<false>, kThreads, sizeof(FusedShared));
        cudaOccupancyMaxActiveBlocksPerMultiprocessor(&c, encode_fused_kernel<true>, kThreads, sizeof(FusedSharedCompact));
        g_raw_ctas_per_sm = a > 0 ? a : 1;
        g_fused_ctas_per_sm = b > 0 ? b : 1;
        g_compact_ctas_per_sm = c > 0 ? c : 1;
    }
    const int per_sm = mode == kEncodeRaw ? g_raw_ctas_per_sm : g_fused_ctas_per_sm;
    unsigned long long cap = (unsigned long long)sm_count * per_sm;
    unsigned grid = (unsigned)(jb.total_tiles < cap ? jb.total_tiles : cap);
    ++g_launches;
    if (mode == kEncodeRaw)
        return launch_k(encode_raw_kernel, dim3(grid), dim3(kThreads), sizeof(EncodeShared), st, jb, ws, host_params, device_params ? 1 : 0);
    // a fused launch whose tiles fit the device at once, but not at the persistent kernel's occupancy, runs as one
    // tile per CTA on the compact instance (no second wave of tiles behind the first)
    const unsigned long long compact_cap = (unsigned long long)sm_count * g_compact_ctas_per_sm;
    if ((jb.total_tiles > cap || compact_mode() == 2) && jb.total_tiles <= compact_cap && compact_mode() != 0)
        return launch_k<false>(encode_fused_kernel<true>, dim3((unsigned)jb.total_tiles), dim3(kThreads), sizeof(FusedSharedCompact), st, jb, ws);
    return launch_k<false>(encode_fused_kernel<false>, dim3(grid), dim3(kThreads), sizeof(FusedShared), st, jb, ws);
}

cudaError_t launch_decode(const JobBatch& jb, const Workspace& ws, int sm_count, cudaStream_t st)
{
    if (jb.total_tiles == 0) return cudaSuccess;
    if (lanes_engine()) {
        ++g_launches;
        return launch_decode_lanes(jb, ws, sm_count, st);
    }
    if (g_decode_ctas_per_sm == 0) {
        int a = 0;
        cudaOccupancyMaxActiveBlocksPerMultiprocessor(&a, decode_kernel, kThreads, 0);
        g_decode_ctas_per_sm = a > 0 ? a : 1;
    }
    unsigned long long cap = (unsigned long long)sm_count * g_decode_ctas_per_sm;
    unsigned grid = (unsigned)(jb.total_tiles < cap ? jb.total_tiles : cap);
    ++g_launches;
    return launch_k(decode_kernel, dim3(grid), dim3(kThreads), 0, st, jb, ws);
}

cudaError_t launch_copy(const CopyBatch& cb, const Workspace& ws, int sm_count, cudaStream_t st)
{
    if (cb.count <= 0) return cudaSuccess;
    unsigned gx = (unsigned)((sm_count * 4 + cb.count - 1) / cb.count);
    ++g_launches;
    return launch_k(copy_kernel, dim3(gx ? gx : 1, cb.count), dim3(256), 0, st, cb, ws);
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
    static int per_sm = 0;     // one wave of resident CTAs, each striding over the arrays
    if (per_sm == 0) {
        int a = 0;
        cudaOccupancyMaxActiveBlocksPerMultiprocessor(&a, quality_kernel, 256, 0);
        per_sm = a > 0 ? a : 1;
    }
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

cudaError_t launch_copy_chain(const ChainBatch& cb, const Workspace& ws, int sm_count, cudaStream_t st)
{
    if (cb.count <= 0 || cb.hops == 0) return cudaSuccess;
    unsigned gx = (unsigned)((sm_count * 4 + cb.count - 1) / cb.count);
    ++g_launches;
    return launch_k(copy_chain_kernel, dim3(gx ? gx : 1, cb.count), dim3(256), 0, st, cb, ws);
}

}  // namespace zccl
