// Binary64 input on the lane-per-block decomposition: included by zccl_codec.cu inside its unnamed namespace, after
// the binary32 kernels whose back ends (bit-matrix transposes, plane loads, blob windows, the placement) it shares.
//
// What differs from binary32 is the way in and the way out.  In: q = rint(fl64(x * r)) comes from one multiplication and
// one addition of 1.5 * 2^52, whose sum carries q in two's complement in its low mantissa word for every |x r| < 2^51;
// deltas, magnitudes and signs are 32-bit integer work from there on (no precision caveat: the codes are exact over
// the whole range |q| < 2^30, which is checked on the exponent bits of x r).  Out: x' = fl64(q * s) with q made a
// binary64 by the same device backwards (the word q ^ 2^31 under the exponent of 2^52, minus 2^52 + 2^31).
//
// A round is still 32 blocks = 1024 elements, now 8 KiB: the array is described to the copy engine as rows of 16
// doubles (128 bytes, the widest row the 128-byte swizzle takes), a round is a box of 64 rows, and lane l owns rows
// 2 l and 2 l + 1.  Chunk c (16 bytes = two doubles) of row t sits at chunk c ^ (t & 7) of that row.  Kernels here
// take one array per launch; one that does not start on a 16-byte boundary is loaded with plain accesses.

constexpr double kMagic52 = 6755399441055744.0;         // 1.5 * 2^52
constexpr double kIntBias = 4503601774854144.0;         // 2^52 + 2^31
constexpr uint32_t kRangeHi = 0x41D00000u;              // high word of 2^30: |t| < 2^30 <=> (hi(t) & 0x7FFFFFFF) < kRangeHi
constexpr int kRowsPerRound64 = 64;                     // rows of 16 doubles
constexpr int kStages64 = 3;

// Byte offset, inside a lane's pair of rows, of the lane's 16-byte chunk k (k = 0 .. 15: elements 2 k and 2 k + 1 of its
// block); sw0 = (2 lane) & 7 is the swizzle of the first row, sw0 | 1 that of the second.
__device__ __forceinline__ uint32_t pair_chunk_byte(uint32_t k, uint32_t sw0) { return (16u * k) ^ ((sw0 | (k >> 3)) << 4); }

// Integer pass over the block in this lane's two rows of a stage: deltas of the codes against the code of the
// element in front (xprev), magnitudes packed 32 / N to a word for the N-bit transpose (word i, field h = element
// N h + i; N = 32: one magnitude per word), OR of the magnitudes, sign word, and the largest high word of |x r| (the
// range check).
template <int N>
struct BlockPack64 {
    uint32_t w[N];
    uint32_t sign, orb, hi_max;
};
template <int N>
__device__ __forceinline__ void block_pass_f64(const char* rows, uint32_t sw0, double xprev, double r, BlockPack64<N>& o)
{
    const double tp = __dmul_rn(xprev, r);
    uint32_t qp = (uint32_t)__double2loint(__dadd_rn(tp, kMagic52));
    uint32_t hm = (uint32_t)__double2hiint(tp) & 0x7FFFFFFFu;
    uint32_t orb = 0, sg = 0;
#pragma unroll
    for (int i = 0; i < N; ++i) o.w[i] = 0;
#pragma unroll 1
    for (uint32_t g = 0; g < 32u / N; ++g) {
#pragma unroll
        for (int q = 0; q < N / 2; ++q) {
            const double2 v = *reinterpret_cast<const double2*>(rows + pair_chunk_byte(g * (N / 2) + q, sw0));
            const double xs[2] = {v.x, v.y};
#pragma unroll
            for (int e = 0; e < 2; ++e) {
                const double t = __dmul_rn(xs[e], r);
                hm = max(hm, (uint32_t)__double2hiint(t) & 0x7FFFFFFFu);
                const uint32_t qq = (uint32_t)__double2loint(__dadd_rn(t, kMagic52));
                const int32_t dd = (int32_t)(qq - qp);
                qp = qq;
                const uint32_t m = (uint32_t)abs(dd);
                orb |= m;
                sg = __funnelshift_l((uint32_t)dd, sg, 1);                     // sign of element j ends up in bit 31 - j
                if (N == 32) o.w[2 * q + e] = m;
                else o.w[2 * q + e] = prmt(o.w[2 * q + e], m, N == 8 ? 0x4321u : 0x5432u);
            }
        }
    }
    o.sign = __brev(sg);
    o.orb = orb;
    o.hi_max = hm;
}

// One round of the encoder's back end for binary64, in place: the block in this lane's two rows of `stage` becomes
// the lane's share of the round's slot image in the same stage (code-length byte `lane`, payload from word 8).
// One width class N (bits per packed magnitude) for the whole warp.  Returns 0 when done (pay_words = the round's
// payload words, width = the class the round needed: 0, 1, 2 for 8, 16, 32); otherwise nothing was stored: 1 when some
// |x r| >= 2^30 (the general route then reports it), 3 (`mid` not called) when a lane's code is longer than N.  `mid` is
// called once, by all lanes, when the rows have been read.
template <int N, class Mid>
__device__ __forceinline__ int encode_round_f64_n(double* stage, uint32_t sw0, double xprev, double r, uint32_t& pay_words, int& width, int lane,
                                                  Mid&& mid)
{
    BlockPack64<N> a;
    block_pass_f64<N>(reinterpret_cast<const char*>(stage) + 256 * lane, sw0, xprev, r, a);
    const bool beyond = a.hi_max >= kRangeHi;
    const uint32_t L = code_length(a.orb);
    if (N < 32 && __any_sync(kFull, L > (uint32_t)N)) return 3;
    const uint32_t nw = L ? L + 1u : 0u;
    const uint32_t incl = warp_incl_scan(nw, lane);
    const uint32_t round_total = __shfl_sync(kFull, incl, 31);
    mid();
    if (__any_sync(kFull, beyond)) return 1;
    __syncwarp();   // every lane has read its rows for the last time: the slot image may lie over the stage
    uint32_t* img = reinterpret_cast<uint32_t*>(stage);
    if (L) {
        uint32_t* dst = img + 8 + (incl - nw);
        dst[0] = a.sign;
        bit_transpose<N>(a.w);
#pragma unroll
        for (int k = 0; k < (N < 31 ? N : 31); ++k)
            if ((uint32_t)k < L) dst[1 + k] = a.w[k];
    }
    reinterpret_cast<unsigned char*>(img)[lane] = (unsigned char)L;
    pay_words = round_total;
    width = __any_sync(kFull, L > 16u) ? 2 : __any_sync(kFull, L > 8u) ? 1 : 0;
    return 0;
}
// The widest class out of line: rare on smooth data, and its 32 words would otherwise set the kernel's register count.
// (No hook here: a closure handed to an out-of-line function would force what it captures into local memory.)
struct WideResult { int rc; uint32_t pay_words; int width; };
__device__ __noinline__ WideResult encode_round_f64_wide(double* stage, uint32_t sw0, double xprev, double r, int lane)
{
    WideResult w;
    w.pay_words = 0; w.width = 2;
    w.rc = encode_round_f64_n<32>(stage, sw0, xprev, r, w.pay_words, w.width, lane, [] {});
    return w;
}
// Starts with the class the round before needed and widens as long as a lane's code does not fit.
template <class Mid>
__device__ __forceinline__ int encode_round_f64(double* stage, uint32_t sw0, double xprev, double r, uint32_t& pay_words, int& width, int lane,
                                                Mid&& mid)
{
    if (width == 0) {
        const int rc = encode_round_f64_n<8>(stage, sw0, xprev, r, pay_words, width, lane, mid);
        if (rc != 3) return rc;
    }
    if (width <= 1) {
        const int rc = encode_round_f64_n<16>(stage, sw0, xprev, r, pay_words, width, lane, mid);
        if (rc != 3) return rc;
    }
    mid();
    const WideResult w = encode_round_f64_wide(stage, sw0, xprev, r, lane);
    if (w.rc == 0) { pay_words = w.pay_words; width = w.width; }
    return w.rc;
}

// General route for one round of a binary64 tile: any code length, ragged ends, straight from global memory into the
// round's slot, conversions by the definition itself.  Compact rather than fast.
__device__ __noinline__ uint32_t encode_round_general_f64(const double* __restrict__ xt, uint32_t len, uint32_t rd, double r, uint32_t* __restrict__ slot,
                                                          uint32_t* round_words, int32_t* outlier, unsigned long long* group_words, int lane)
{
    uint32_t status = 0;
    const uint32_t nb = (len + kBlock - 1) / kBlock;
    const uint32_t bi = 32u * rd + (uint32_t)lane;
    const uint32_t last = len - 1;
    uint32_t L = 0, sgw = 0;
    uint32_t m[32];
    if (bi < nb) {
        const uint32_t e0 = 32u * bi;
        const uint32_t ep = e0 ? e0 - 1u : 0u;
        const double tp = __dmul_rn(__ldg(xt + (ep < last ? ep : last)), r);
        bool out_of_range = !(fabs(tp) < 1073741824.0);   // also true for a NaN
        uint32_t qp = (uint32_t)__double2int_rn(tp);
        uint32_t sg = 0, ob = 0;
#pragma unroll
        for (int j = 0; j < 32; ++j) {
            const uint32_t e = e0 + (uint32_t)j;
            const double t = __dmul_rn(__ldg(xt + (e < last ? e : last)), r);
            out_of_range = out_of_range || !(fabs(t) < 1073741824.0);
            const uint32_t q = (uint32_t)__double2int_rn(t);
            const int32_t dd = (int32_t)(q - qp);
            qp = q;
            const uint32_t sm = (uint32_t)(dd >> 31);
            m[j] = (((uint32_t)dd ^ sm) - sm) & 0x7FFFFFFFu;   // |delta|; the mask only matters after a range error
            ob |= m[j];
            sg = __funnelshift_l((uint32_t)dd, sg, 1);
        }
        if (out_of_range) status |= kStRange;
        L = code_length(ob);
        sgw = __brev(sg);
        bit_transpose<32>(m);
    }
    const uint32_t nw = L ? L + 1u : 0u;
    const uint32_t incl = warp_incl_scan(nw, lane);
    reinterpret_cast<unsigned char*>(slot)[lane] = (unsigned char)L;
    if (L) {
        uint32_t* d = slot + 8 + (incl - nw);
        d[0] = sgw;
#pragma unroll
        for (int k = 0; k < 31; ++k)
            if ((uint32_t)k < L) d[1 + k] = m[k];
    }
    if (lane == 31) { *round_words = incl; atomicAdd(group_words, (unsigned long long)incl); }
    if (rd == 0 && lane == 0) *outlier = __double2int_rn(__dmul_rn(__ldg(xt), r));
    return status;
}

// A full round of an array that the copy engine cannot take (not on a 16-byte boundary): plain coalesced loads into the
// stage's layout.
__device__ __noinline__ void load_round_plain_f64(double* stage, const double* __restrict__ xr, int lane)
{
#pragma unroll 4
    for (uint32_t k = 0; k < 32u; ++k) {
        const uint32_t e = 32u * k + (uint32_t)lane;
        *reinterpret_cast<double*>(reinterpret_cast<char*>(stage) + stage_chunk_byte(e >> 4, (e & 15u) >> 1) + 8u * (e & 1u)) = __ldg(xr + e);
    }
}

struct alignas(1024) RoundWarpShared64 {
    double stage[kStages64][kRound];           // 8 KiB each, on 1024-byte boundaries; a round is encoded in place and leaves from here
    alignas(16) double front[kStages64][2];    // the two elements in front of each stage's round
    alignas(8) unsigned long long bar[kStages64];
};

// Step 1 of a binary64 compression (step 2 is place_kernel): the CTA's four warps take the four rounds of a tile, the
// CTAs take the tiles in turn; a full round comes in by one tensor copy (one round ahead with two stages), is encoded
// in place and leaves by one bulk store to its slot, exactly as in encode_rounds_kernel; partial rounds (the end of
// the array) take the general route.
__global__ void __launch_bounds__(kCodecThreads, kStages64 == 2 ? 3 : 2) encode_rounds_f64_kernel(const double* __restrict__ x, unsigned long long n, uint32_t tiles,
                                                                             const __grid_constant__ CUtensorMap map, int mapped, Workspace ws,
                                                                             ParamsF64 hp, int use_dev_params)
{
    pdl_enter();
    extern __shared__ __align__(16) unsigned char smem_raw[];
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    RoundWarpShared64& sh = reinterpret_cast<RoundWarpShared64*>(smem_raw + ((1024u - (smem_u32(smem_raw) & 1023u)) & 1023u))[warp];
    uint32_t status = 0;
    ParamsF64 prm = hp;
    if (use_dev_params) prm = *ws.params64;
    const double r = prm.r;
    if (lane == 0) {
#pragma unroll
        for (int k = 0; k < kStages64; ++k) mbar_init(&sh.bar[k], 1);
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    __syncwarp();

    const unsigned long long G = gridDim.x;
    const uint32_t rd = (uint32_t)warp, e0 = rd * (uint32_t)kRound;
    const uint32_t sw0 = (2u * (uint32_t)lane) & 7u;
    auto tile_len = [&](unsigned long long t) -> uint32_t {
        if (t >= tiles || !prm.valid || n == 0) return 0u;
        const unsigned long long left = n - t * kTile;
        return (uint32_t)(left < (unsigned long long)kTile ? left : (unsigned long long)kTile);
    };
    // Asks for the warp's round of tile t into stage st; completes one phase of the stage's mbarrier whether there is
    // anything to copy or not.
    auto request = [&](unsigned long long t, uint32_t st) {
        if (e0 + (uint32_t)kRound <= tile_len(t)) {
            if (mapped) {
                if (lane == 0) {
                    mbar_expect_tx(&sh.bar[st], kRound * 8 + (rd ? 16u : 0u));
                    asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
                    asm volatile("cp.async.bulk.tensor.2d.shared::cluster.global.tile.mbarrier::complete_tx::bytes [%0], [%1, {%2, %3}], [%4];"
                                 ::"r"(smem_u32(sh.stage[st])), "l"(&map), "r"(0), "r"((int)((uint32_t)t * 256u + rd * (uint32_t)kRowsPerRound64)),
                                   "r"(smem_u32(&sh.bar[st])) : "memory");
                    if (rd)
                        asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], 16, [%2];"
                                     ::"r"(smem_u32(sh.front[st])), "l"(x + t * kTile + e0 - 2), "r"(smem_u32(&sh.bar[st])) : "memory");
                }
                return;
            }
            load_round_plain_f64(sh.stage[st], x + t * kTile + e0, lane);
            if (lane == 0 && rd) sh.front[st][1] = __ldg(x + t * kTile + e0 - 1);
            __syncwarp();
        }
        if (lane == 0) mbar_arrive(&sh.bar[st]);
    };

    unsigned long long t = blockIdx.x;
#pragma unroll
    for (int k = 0; k + 1 < kStages64; ++k) request(t + (unsigned long long)k * G, (uint32_t)k);
    uint32_t st = 0, phase = 0;
    int width = 0;   // the class the warp's last round needed
    while (t < tiles) {
        const uint32_t len = tile_len(t);
        const uint32_t u = 4u * (uint32_t)t + rd;
        const uint32_t nb = (len + kBlock - 1) / kBlock;
        if (!mbar_wait(&sh.bar[st], phase)) status |= kStTimeout;
        // the stage the request goes to was encoded in place and sent off one step ago: the copy engine has to be through
        // with reading it
        auto mid = [&]() {
            if (lane == 0) asm volatile("cp.async.bulk.wait_group.read 0;" ::: "memory");
            __syncwarp();
            request(t + (unsigned long long)(kStages64 - 1) * G, st == 0 ? (uint32_t)kStages64 - 1u : st - 1u);
        };
        if (32u * rd < nb) {
            uint32_t* slot = ws.slots + (size_t)u * kRoundSlotWords;
            const uint32_t gslot = (uint32_t)(t >> 5);
            int rc = 1;
            uint32_t pay_words = 0;
            double* stage = sh.stage[st];
            if (e0 + (uint32_t)kRound <= len) {
                const double first = stage[0];
                const double xprev = lane ? *reinterpret_cast<const double*>(reinterpret_cast<const char*>(stage) + 256 * lane - 128 +
                                                                             ((7u ^ ((2u * (uint32_t)lane - 1u) & 7u)) << 4) + 8)
                                          : (rd ? sh.front[st][1] : first);
                rc = encode_round_f64(stage, sw0, xprev, r, pay_words, width, lane, mid);
                if (rc == 0) {
                    __syncwarp();   // the words written by all lanes are visible to lane 0's store
                    if (lane == 0) {
                        const uint32_t bytes = (32u + 4u * pay_words + 15u) & ~15u;
                        asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
                        asm volatile("cp.async.bulk.global.shared::cta.bulk_group [%0], [%1], %2;" ::"l"(slot), "r"(smem_u32(stage)), "r"(bytes) : "memory");
                        asm volatile("cp.async.bulk.commit_group;" ::: "memory");
                        ws.round_words[u] = pay_words;
                        atomicAdd(ws.group_acc + gslot, (unsigned long long)pay_words);
                        if (rd == 0) ws.outliers[t] = __double2loint(__dadd_rn(__dmul_rn(first, r), kMagic52));
                    }
                }
            } else {
                mid();
            }
            if (rc != 0)
                status |= encode_round_general_f64(x + t * kTile, len, rd, r, slot, ws.round_words + u, ws.outliers + t, ws.group_acc + gslot, lane);
        } else {
            mid();
            if (lane == 0) ws.round_words[u] = 0;   // a round beyond the tile's last block, or a tile without elements
        }
        t += G;
        st = st == (uint32_t)kStages64 - 1u ? 0u : st + 1u;
        if (st == 0) phase ^= 1u;
    }
    if (lane == 0) asm volatile("cp.async.bulk.wait_group 0;" ::: "memory");   // the stores have read shared memory and are complete
    if (status) atomicOr(ws.status, status);
}

// ------------------------------------------------------------------------------------------------ binary64, decompress

struct StreamInfo64 {
    unsigned long long n;
    uint32_t nT;
    double s;
    bool ok;
};
__device__ __forceinline__ StreamInfo64 read_header_f64(const uint32_t* in, unsigned long long cap_bytes)
{
    StreamInfo64 h;
    h.ok = false; h.n = 0; h.nT = 0; h.s = 1.0;
    if (cap_bytes < (unsigned)kHeaderBytes) return h;
    const uint32_t magic = ldg_u32(in + 0), ver = ldg_u32(in + 1);
    const unsigned long long n = (unsigned long long)ldg_u32(in + 2) | ((unsigned long long)ldg_u32(in + 3) << 32);
    const double s = __hiloint2double((int)ldg_u32(in + 5), (int)ldg_u32(in + 4));
    const uint32_t T = ldg_u32(in + 6), nT = ldg_u32(in + 7);
    if (magic != kMagic || ver != kVersionF64 || T != (uint32_t)kTile) return h;
    if ((n + kTile - 1) / kTile != nT) return h;
    if (cap_bytes < (unsigned long long)kHeaderBytes + 4ull * nT) return h;
    if (!(s > 0.0) || !isfinite(s)) return h;
    h.n = n; h.nT = nT; h.s = s; h.ok = true;
    return h;
}

// A code as a binary64, exactly: the word q ^ 2^31 under the exponent of 2^52 is 2^52 + 2^31 + q.
__device__ __forceinline__ double code_to_double(int32_t q)
{
    return __dsub_rn(__hiloint2double(0x43300000, (int)((uint32_t)q ^ 0x80000000u)), kIntBias);
}

// The lane's 32 elements from the transposed words (word i, field h = magnitude of element N h + i) as values in the
// lane's two rows of a stage: field, sign, running code (32-bit integers), one conversion and one multiplication.
template <int N>
__device__ __forceinline__ void expand_block_f64(const uint32_t (&w)[N], uint32_t sign, int32_t code_in_front, double s, char* rows, uint32_t sw0)
{
    int32_t run = code_in_front;
    uint32_t sel = N == 8 ? 0x4440u : 0x4410u;   // byte (pair) h of a word, zero above it
#pragma unroll 1
    for (uint32_t h = 0; h < 32u / N; ++h) {
#pragma unroll
        for (int q = 0; q < N / 2; ++q) {
            double o[2];
#pragma unroll
            for (int e = 0; e < 2; ++e) {
                const int i = 2 * q + e;
                const int32_t m = (int32_t)prmt(w[i], 0u, sel);
                run += ((sign >> i) & 1u) ? -m : m;
                o[e] = __dmul_rn(code_to_double(run), s);
            }
            *reinterpret_cast<double2*>(rows + pair_chunk_byte(h * (N / 2) + (uint32_t)q, sw0)) = make_double2(o[0], o[1]);
        }
        sign >>= N;
        sel += N == 8 ? 0x0001u : 0x0022u;
    }
}

// One round of a binary64 tile by the general route: any code length.  Arguments as for decode_round_f64.
__device__ __noinline__ void decode_round_general_f64(const uint32_t* blob, uint32_t padw, uint32_t L, uint32_t* pay_off_io, int32_t* code_io,
                                                      double s, double* stage, int lane)
{
    const uint32_t nw = L ? L + 1u : 0u;
    const uint32_t incl = warp_incl_scan(nw, lane);
    const uint32_t* pay = blob + 1 + padw + *pay_off_io + (incl - nw);
    *pay_off_io += __shfl_sync(kFull, incl, 31);
    const uint32_t sign = L ? pay[0] : 0u;
    uint32_t w[32];
    int32_t total = 0;
#pragma unroll
    for (int k = 0; k < 32; ++k) {
        w[k] = (uint32_t)k < L ? pay[1 + k] : 0u;
        total += (__popc(w[k]) - 2 * __popc(w[k] & sign)) << k;
    }
    int32_t inc = total;
#pragma unroll
    for (int d = 1; d < 32; d <<= 1) {
        const int32_t v = __shfl_up_sync(kFull, inc, d);
        if (lane >= d) inc += v;
    }
    bit_transpose<32>(w);
    int32_t run = *code_io + inc - total;
    *code_io += __shfl_sync(kFull, inc, 31);
    char* rows = reinterpret_cast<char*>(stage) + 256 * lane;
    const uint32_t sw0 = (2u * (uint32_t)lane) & 7u;
#pragma unroll
    for (int j = 0; j < 32; ++j) {
        run += ((sign >> j) & 1u) ? -(int32_t)w[j] : (int32_t)w[j];
        *reinterpret_cast<double*>(rows + pair_chunk_byte((uint32_t)j >> 1, sw0) + 8u * (j & 1)) = __dmul_rn(__int2double_rn(run), s);
    }
}

// One round of a binary64 tile: blocks 32 rd + lane; blob: the tile's words (or a window over them), pay_off: payload
// words of the rounds before, code: the code in front of the round.  Leaves the values in `stage`, which `ready` (called
// once by all lanes, after the planes are read and before the first value is stored) makes sure is free.
template <class Ready>
__device__ __forceinline__ void decode_round_f64(const uint32_t* blob, uint32_t padw, uint32_t L, uint32_t& pay_off, int32_t& code, double s,
                                                 double* stage, int lane, Ready&& ready)
{
    if (__any_sync(kFull, L > 16u)) {
        ready();
        decode_round_general_f64(blob, padw, L, &pay_off, &code, s, stage, lane);
        return;
    }
    const uint32_t nw = L ? L + 1u : 0u;
    const uint32_t incl = warp_incl_scan(nw, lane);
    const uint32_t* pay = blob + 1 + padw + pay_off + (incl - nw);
    pay_off += __shfl_sync(kFull, incl, 31);
    char* rows = reinterpret_cast<char*>(stage) + 256 * lane;
    const uint32_t sw0 = (2u * (uint32_t)lane) & 7u;
    uint32_t sign;
    int32_t total;
    if (!__any_sync(kFull, L > 8u)) {
        uint32_t w[8];
        total = load_planes<8>(pay, L, sign, w);
        int32_t inc = total;
#pragma unroll
        for (int d = 1; d < 32; d <<= 1) {
            const int32_t v = __shfl_up_sync(kFull, inc, d);
            if (lane >= d) inc += v;
        }
        bit_transpose<8>(w);
        ready();
        expand_block_f64<8>(w, sign, code + inc - total, s, rows, sw0);
        code += __shfl_sync(kFull, inc, 31);
    } else {
        uint32_t w[16];
        total = load_planes<16>(pay, L, sign, w);
        int32_t inc = total;
#pragma unroll
        for (int d = 1; d < 32; d <<= 1) {
            const int32_t v = __shfl_up_sync(kFull, inc, d);
            if (lane >= d) inc += v;
        }
        bit_transpose<16>(w);
        ready();
        expand_block_f64<16>(w, sign, code + inc - total, s, rows, sw0);
        code += __shfl_sync(kFull, inc, 31);
    }
}

// `count` elements of a stage to global memory, coalesced (ragged ends).
__device__ __noinline__ void store_round_ragged_f64(double* __restrict__ y, const double* stage, uint32_t count, int lane)
{
#pragma unroll 4
    for (uint32_t k = 0; k < 32u; ++k) {
        const uint32_t e = 32u * k + (uint32_t)lane;
        const uint32_t row = e >> 4, chunk = (e & 15u) >> 1;
        if (e < count) y[e] = *reinterpret_cast<const double*>(reinterpret_cast<const char*>(stage) + stage_chunk_byte(row, chunk) + 8u * (e & 1u));
    }
}

struct alignas(1024) DecWarpShared64 {
    double out[kRound];                     // one 8 KiB stage: a round's planes are read and transposed while the store of the round before drains it
    alignas(16) uint32_t blob[kDecBlobWords];
    alignas(8) unsigned long long bar;
};

// A warp decodes a tile of its own in four rounds, as decode_tiles_kernel does: blob staged by bulk copies (a window
// at a time when it is larger than the buffer, the next tile's as soon as this tile's last round is decoded), values
// into the stage, one tensor store per full round (`mapped`: y starts on a 16-byte boundary and has a map), plain
// coalesced stores otherwise.
__global__ void __launch_bounds__(kCodecThreads, 4) decode_tiles_f64_kernel(const uint32_t* __restrict__ in, unsigned long long in_cap,
                                                                            double* __restrict__ y, unsigned long long y_cap, uint32_t tiles,
                                                                            const __grid_constant__ CUtensorMap map, int mapped, Workspace ws)
{
    pdl_enter();
    extern __shared__ __align__(16) unsigned char smem_raw[];
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    DecWarpShared64& sh = reinterpret_cast<DecWarpShared64*>(smem_raw + ((1024u - (smem_u32(smem_raw) & 1023u)) & 1023u))[warp];
    uint32_t status = 0;
    if (lane == 0) {
        mbar_init(&sh.bar, 1);
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    __syncwarp();
    const StreamInfo64 h = read_header_f64(in, in_cap);
    if (!h.ok || h.n > y_cap) {
        if (tid == 0 && blockIdx.x == 0) atomicOr(ws.status, h.ok ? kStCapacity : kStBadStream);
        return;
    }
    uint32_t fills = 0;   // bulk copies completed into the blob buffer (phase parity of its mbarrier)
    const unsigned long long blob0 = (unsigned long long)kHeaderWords + h.nT;
    const uint32_t last_tile = h.nT < tiles ? h.nT : tiles;

    // The blob of tile t, from the index alone; the front of its 16-byte-aligned cover is requested into the blob buffer
    // when the cover lies inside the readable bytes.  Uniform over the warp.
    auto request = [&](unsigned long long t) {
        BlobRef br;
        br.ptr = nullptr; br.words = 0; br.staged = false;
        if (t >= last_tile) return br;
        const uint32_t* idx = in + kHeaderWords;
        const uint32_t w_end = ldg_u32(idx + t);
        const uint32_t w_beg = t ? ldg_u32(idx + t - 1) : 0u;
        if (w_end <= w_beg || (blob0 + w_end) * 4ull > in_cap) { br.words = 0xFFFFFFFFu; return br; }   // marks a damaged index
        br.ptr = in + blob0 + w_beg;
        br.words = w_end - w_beg;
        const uintptr_t a_end = ((uintptr_t)(br.ptr + br.words) + 15) & ~(uintptr_t)15;
        if (a_end - (uintptr_t)in <= (uintptr_t)in_cap) {   // the copies may read up to the boundary behind the blob
            if (lane == 0) window_request(br, 0, sh.blob, &sh.bar);
            br.staged = true;
        }
        return br;
    };

    const unsigned long long stride = (unsigned long long)gridDim.x * kCodecWarps;
    unsigned long long t = (unsigned long long)blockIdx.x * kCodecWarps + (unsigned long long)warp;
    BlobRef cur = request(t);
    while (t < last_tile) {
        const unsigned long long tn = t + stride;
        BlobRef nxt;
        nxt.ptr = nullptr; nxt.words = 0; nxt.staged = false;
        bool asked = false;
        auto ask_next = [&]() {
            __syncwarp();   // every lane is done with the blob buffer
            nxt = request(tn);
            asked = true;
        };
        if (cur.staged) {
            if (!mbar_wait(&sh.bar, fills & 1u)) status |= kStTimeout;
            ++fills;
        }
        if (cur.words == 0xFFFFFFFFu) status |= kStBadStream;
        else if (cur.ptr) {
            const unsigned long long start = t * kTile;
            const uint32_t len = (uint32_t)((h.n - start < (unsigned long long)kTile) ? (h.n - start) : kTile);
            const uint32_t nb = (len + kBlock - 1) / kBlock, padw = (nb + 3) >> 2;
            BlobWindow win;
            win.base = cur.ptr; win.end = cur.words;
            if (cur.staged) win = window_at(cur, 0, sh.blob);
            if (describe_blob(win.base, cur.words, nb, lane) == 0) status |= kStBadStream;
            else {
                uint32_t pay_off = 0;
                int32_t code = (int32_t)win.base[0];
                const uint32_t lp = lane_code_lengths(win.base, nb, lane);
                const uint32_t rounds = (nb + 31) >> 5;
                for (uint32_t rd = 0; rd < rounds; ++rd) {
                    const uint32_t L = (lp >> (8u * rd)) & 0xFFu;
                    const uint32_t first = 1u + padw + pay_off;
                    if (win.end < cur.words && first + __reduce_add_sync(kFull, L ? L + 1u : 0u) > win.end) {   // the round reaches past the window
                        __syncwarp();
                        if (lane == 0) window_request(cur, first, sh.blob, &sh.bar);
                        if (!mbar_wait(&sh.bar, fills & 1u)) status |= kStTimeout;
                        ++fills;
                        win = window_at(cur, first, sh.blob);
                    }
                    // the stage was handed to a tensor store a round ago
                    auto ready = [&]() {
                        if (lane == 0) asm volatile("cp.async.bulk.wait_group.read 0;" ::: "memory");
                        __syncwarp();
                    };
                    decode_round_f64(win.base, padw, L, pay_off, code, h.s, sh.out, lane, ready);
                    if (rd + 1 == rounds) ask_next();
                    __syncwarp();   // the stage's rows, written by all lanes, are visible
                    const uint32_t e0 = rd * (uint32_t)kRound;
                    if (mapped && e0 + (uint32_t)kRound <= len) {
                        if (lane == 0) {
                            asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
                            asm volatile("cp.async.bulk.tensor.2d.global.shared::cta.tile.bulk_group [%0, {%1, %2}], [%3];"
                                         ::"l"(&map), "r"(0), "r"((int)((uint32_t)t * 256u + rd * (uint32_t)kRowsPerRound64)), "r"(smem_u32(sh.out)) : "memory");
                            asm volatile("cp.async.bulk.commit_group;" ::: "memory");
                        }
                    } else {
                        store_round_ragged_f64(y + start + e0, sh.out, len - e0 < (uint32_t)kRound ? len - e0 : (uint32_t)kRound, lane);
                        __syncwarp();   // the stage is read before the next round overwrites it
                    }
                }
            }
        }
        if (!asked) ask_next();
        cur = nxt;
        t = tn;
    }
    if (lane == 0) asm volatile("cp.async.bulk.wait_group 0;" ::: "memory");
    if (status) atomicOr(ws.status, status);
}
