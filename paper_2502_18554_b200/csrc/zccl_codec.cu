// fZ-light codec kernels for sm_100a: encoder, decoder and the fused decode + reduce + encode hop.
//
// Work decomposition: ONE LANE OWNS ONE 32-ELEMENT BLOCK.  A warp works on a 4096-element tile of its own in four
// rounds of 32 blocks (1024 elements); lane l of a round holds the 32 consecutive elements of block l in registers.
// Everything the format asks of a block then happens inside one thread, with no shuffle, vote or barrier:
//   * quantise and 1-D Lorenzo delta: fp32 on the FMA pipe (t + 1.5 * 2^23 rounds to nearest even, deltas of two
//     such values are exact, |delta| + 2^23 has the magnitude in its mantissa);
//   * code length: OR of the 32 magnitudes, one count-leading-zeros;
//   * bit planes: the magnitudes are packed four (code lengths up to 8), two (up to 16) or one to a word and an
//     in-register bit-matrix transpose (3, 4 or 5 stages of shift + bit-select pairs) turns them into plane words;
//   * sign word: one funnel shift per element.
// A warp needs its neighbours only for the prefix sum of the blocks' sizes (one shuffle scan per round) and, when it
// decodes, of the blocks' delta sums.  Warps never wait for each other inside a CTA: there is no __syncthreads in
// the tile loops.
//
// Memory.  A lane wants 128 consecutive bytes per block while global accesses must be contiguous across the warp,
// so rounds go through shared memory: the warp copies 4 KiB with 16-byte asynchronous copies (cp.async, no
// registers, one round ahead) into a stage whose 16-byte chunks are XOR-swizzled by the row number, so that the
// copy, the lanes' 128-bit row reads and (decoder) the row writes are all free of bank conflicts.  A tile's blob is
// assembled in the warp's shared memory and moved to the stream once its position is known.
//
// Placement.  Tiles are handed out in order by a device-wide counter, so every tile before a given one is already
// owned by a running warp.  A warp publishes its tile's size as soon as it is known and finds its position by a
// decoupled look-back over the 8-byte states of the tiles in front of it (32 at a time, one per lane), stopping at
// the first one that carries an inclusive prefix; states are validated by a launch counter instead of being cleared.
// Every wait is bounded and reports through the status word instead of hanging.
#include "zccl_device.cuh"

#include <mutex>

namespace zccl {
#ifdef ZCCL_TRACE
__device__ unsigned long long g_trace[16];
__device__ unsigned long long g_rec[4096 * 8];
__device__ __forceinline__ unsigned long long gtime() { unsigned long long v; asm volatile("mov.u64 %0, %globaltimer;" : "=l"(v)); return v; }
#define TR_DECL unsigned long long tr_t0 = clock64(), tr_acc[8] = {0,0,0,0,0,0,0,0}; const unsigned long long tr_g0 = gtime()
#define TR_MARK(k) do { const unsigned long long tr_now = clock64(); tr_acc[k] += tr_now - tr_t0; tr_t0 = tr_now; } while (0)
#define TR_FLUSH do { if (lane == 0) { for (int k = 0; k < 8; ++k) atomicAdd(&g_trace[k], tr_acc[k]); atomicAdd(&g_trace[8], 1ull); const unsigned long long g1 = gtime(); atomicMin(&g_trace[9], tr_g0); atomicMax(&g_trace[10], tr_g0); atomicMin(&g_trace[11], g1); atomicMax(&g_trace[12], g1); atomicAdd(&g_trace[13], g1 - tr_g0); } } while (0)
#else
#define TR_DECL
#define TR_MARK(k)
#define TR_FLUSH
#endif
namespace {

constexpr int kCodecWarps = 4;                        // warps per CTA, each with tiles of its own
constexpr int kCodecThreads = 32 * kCodecWarps;
constexpr int kRound = 32 * kBlock;                   // elements per round: one block per lane
constexpr int kRoundsPerTile = kTile / kRound;
constexpr int kLWords = kBlocksPerTile / 4;           // code-length words of a full tile
constexpr int kBlobHeadWords = 1 + kLWords;           // outlier + code lengths
constexpr int kMaxPayWords = kBlocksPerTile * 32;     // every block at code length 31: sign word + 31 planes

// ------------------------------------------------------------------------------------------------ small pieces

__device__ __forceinline__ void cp_async16(uint32_t smem_addr, const void* g)
{
    asm volatile("cp.async.cg.shared.global [%0], [%1], 16;" ::"r"(smem_addr), "l"(g) : "memory");
}
__device__ __forceinline__ void cp_async_commit() { asm volatile("cp.async.commit_group;" ::: "memory"); }
template <int N>
__device__ __forceinline__ void cp_async_wait()
{
    asm volatile("cp.async.wait_group %0;" ::"n"(N) : "memory");
}

__device__ __forceinline__ uint32_t warp_incl_scan(uint32_t v, int lane)
{
#pragma unroll
    for (int d = 1; d < 32; d <<= 1) {
        const uint32_t t = __shfl_up_sync(kFull, v, d);
        if (lane >= d) v += t;
    }
    return v;
}

// In-register bit-matrix transpose of N words (N = 8, 16, 32).  Word i holds 32 / N values of N bits each: value
// number N * h + i sits in bits [N h, N h + N).  Afterwards word k holds plane k: bit N * h + i = bit k of that value.
// Each stage exchanges, between words i and i + d, the bits whose in-value position has bit d set against those that
// have it clear: two shifts and two bit-selects per pair.  The transpose is its own inverse.
template <int N>
__device__ __forceinline__ void bit_transpose(uint32_t (&w)[N])
{
#pragma unroll
    for (int d = N / 2; d >= 1; d >>= 1) {
        const uint32_t m = d == 16 ? 0x0000FFFFu : d == 8 ? 0x00FF00FFu : d == 4 ? 0x0F0F0F0Fu : d == 2 ? 0x33333333u : 0x55555555u;
#pragma unroll
        for (int i = 0; i < N; ++i) {
            if (i & d) continue;
            const uint32_t a = w[i], b = w[i + d];
            w[i] = (a & m) | ((b << d) & ~m);
            w[i + d] = ((a >> d) & m) | (b & ~m);
        }
    }
}

// ------------------------------------------------------------------------------------------------ stages

// A stage holds one round: row t = the 32 floats of block t (128 bytes), its 16-byte chunk c stored at chunk
// position c ^ (t & 7) of the row.
__device__ __forceinline__ uint32_t stage_chunk_byte(uint32_t row, uint32_t chunk) { return row * 128u + ((chunk ^ (row & 7u)) << 4); }

// Brings elements [e0, e0 + 1024) of a tile that has `len` elements at xt into a stage.  Full rounds that start on
// a 16-byte boundary are copied asynchronously (the caller commits and waits); others element by element, positions
// beyond the tile's end repeating its last element (so that the padding of the last block has zero deltas).
__device__ __noinline__ void load_round_ragged(float* stage, const float* __restrict__ xt, uint32_t e0, uint32_t len, int lane)
{
    const uint32_t last = len - 1;
#pragma unroll 4
    for (int k = 0; k < 32; ++k) {
        const uint32_t e = e0 + 32u * k + (uint32_t)lane;
        const float v = __ldg(xt + (e < last ? e : last));
        *reinterpret_cast<float*>(reinterpret_cast<char*>(stage) + stage_chunk_byte(k, (uint32_t)lane >> 2) + 4 * (lane & 3)) = v;
    }
}
// lane_off0 / lane_off1: this lane's byte offset inside the four rows its copies go to, for even / odd copy numbers
__device__ __forceinline__ void load_round(float* stage, const float* __restrict__ xt, uint32_t e0, uint32_t len, int lane, uint32_t lane_off0,
                                           uint32_t lane_off1)
{
    const float* src = xt + e0;
    if (e0 + (uint32_t)kRound <= len && (((uintptr_t)src) & 15u) == 0) {
        const uint32_t sb = smem_u32(stage);
        const char* g = reinterpret_cast<const char*>(src) + 16 * lane;
#pragma unroll
        for (int k = 0; k < 8; ++k) cp_async16(sb + 512u * k + ((k & 1) ? lane_off1 : lane_off0), g + 512 * k);
    } else {
        load_round_ragged(stage, xt, e0, len, lane);
    }
}

// The last element of a row of a stage (the element in front of the next row's block).
__device__ __forceinline__ float read_last_of_row(const float* stage, uint32_t row)
{
    return *reinterpret_cast<const float*>(reinterpret_cast<const char*>(stage) + stage_chunk_byte(row, 7) + 12);
}

// ------------------------------------------------------------------------------------------------ one block, encode

// fp32 pass over the block in this lane's row of a stage: deltas against the element in front (xprev), magnitudes
// packed 32 / N to a word for the N-bit transpose (word i, field h = element N h + i), OR of the magnitude words, sign
// word, and the sum of squares of x * r that tells whether fp32 was exact (below 2^43: every |x r| < 2^21.5).  N = 8
// serves code lengths up to 8, N = 16 up to 16.  The loop over groups of N elements is kept rolled: every word shifts
// down by one field and takes the new magnitude on top, so the body is the same for every group and stays small
// enough for the instruction cache of a scheduler (unrolled, the kernel stalled on instruction fetch).
template <int N>
struct BlockPack {
    uint32_t w[N];
    uint32_t sign, orb;
    float guard;
};
template <int N>
__device__ __forceinline__ void block_pass(const char* row, uint32_t sw, float xprev, float r, BlockPack<N>& o)
{
    const float tp = __fmul_rn(xprev, r);
    float cp = __fadd_rn(tp, kRoundMagic);
    float acc = __fmul_rn(tp, tp);
    uint32_t orb = 0, sg = 0;
#pragma unroll
    for (int i = 0; i < N; ++i) o.w[i] = 0;
#pragma unroll 1
    for (uint32_t g = 0; g < 32u / N; ++g) {
#pragma unroll
        for (int q = 0; q < N / 4; ++q) {
            const float4 v = *reinterpret_cast<const float4*>(row + ((16u * (g * (N / 4) + q)) ^ sw));
            const float xs[4] = {v.x, v.y, v.z, v.w};
#pragma unroll
            for (int e = 0; e < 4; ++e) {
                const float t = __fmul_rn(xs[e], r);
                acc = __fmaf_rn(t, t, acc);
                const float c = __fadd_rn(t, kRoundMagic);
                const float d = __fsub_rn(c, cp);
                cp = c;
                const uint32_t m = __float_as_uint(__fadd_rn(fabsf(d), kTwo23));   // bits 0..22: |delta|
                orb |= m;
                sg = __funnelshift_l(__float_as_uint(d), sg, 1);                  // sign of element j ends up in bit 31 - j
                o.w[4 * q + e] = prmt(o.w[4 * q + e], m, N == 8 ? 0x4321u : 0x5432u);
            }
        }
    }
    o.sign = __brev(sg);
    o.orb = orb & 0x007FFFFFu;
    o.guard = acc;
}

__device__ __forceinline__ uint32_t code_length(uint32_t orb) { return 32u - (uint32_t)__clz((int)orb); }

// Largest |x r| of a block (the rare recheck behind the precision warning).
__device__ __forceinline__ float block_tmax(const char* row, uint32_t sw, float r)
{
    float tm = 0.0f;
#pragma unroll 1
    for (uint32_t q = 0; q < 8; ++q) {
        const float4 v = *reinterpret_cast<const float4*>(row + ((16u * q) ^ sw));
        tm = fmaxf(fmaxf(tm, fabsf(__fmul_rn(v.x, r))), fmaxf(fabsf(__fmul_rn(v.y, r)), fmaxf(fabsf(__fmul_rn(v.z, r)), fabsf(__fmul_rn(v.w, r)))));
    }
    return tm;
}

// What the lanes carry from round to round of a tile they encode.
struct EncodeCarry {
    uint32_t pay_used;   // payload words of the rounds so far
    bool wide;           // the round before had a code length above 8: start with the 16-bit pass
};

// One round of the encoder's back end, for the block in this lane's row of a stage (row: its first byte, sw: the
// lane's chunk swizzle; xprev: the element in front of the block).
// Appends the round's payload to the tile's blob in shared memory (word i of the blob at blob[org + sgn * i]) and
// sets the lane's code-length byte.  `active`: the block exists (ragged tiles have fewer than 128).  Returns 0 when
// done; otherwise nothing was stored: 1 when the round is beyond what this path covers (a code length above 16, or
// codes for which fp32 is not exact) and the whole tile has to take the general route, 2 when the blob would
// outgrow `pay_cap` payload words.
__device__ __forceinline__ int encode_round(const char* row, uint32_t sw, float xprev, float r, bool active, uint32_t block_in_tile,
                                            uint32_t lbytes, uint32_t* __restrict__ blob, uint32_t org, int sgn, uint32_t pay_base,
                                            uint32_t pay_cap, EncodeCarry& cy, int lane, uint32_t& status)
{
    BlockPack<8> a;
    BlockPack<16> h;
    uint32_t L = 0, sign = 0;
    float guard = 0.0f;
    bool need16 = cy.wide;   // uniform over the warp
    if (!need16) {
        block_pass<8>(row, sw, xprev, r, a);
        L = code_length(a.orb);
        sign = a.sign;
        guard = a.guard;
        need16 = L > 8u;     // only these lanes run the second pass
    }
    if (need16) {
        block_pass<16>(row, sw, xprev, r, h);
        L = code_length(h.orb);
        sign = h.sign;
        guard = h.guard;
    }
    if (!active) L = 0;
    const bool beyond = !(guard < kGuardExact) || L > 16u;
    const uint32_t nw = L ? L + 1u : 0u;
    const uint32_t incl = warp_incl_scan(nw, lane);
    const uint32_t round_total = __shfl_sync(kFull, incl, 31);
    if (__any_sync(kFull, beyond)) return 1;
    if (cy.pay_used + round_total > pay_cap) return 2;
    if (guard >= kGuardSmall && block_tmax(row, sw, r) > 32768.5f) status |= kStPrecision;
    if (L) {
        uint32_t* dst = blob + ((int)org + sgn * (int)(pay_base + cy.pay_used + (incl - nw)));
        dst[0] = sign;
        if (!cy.wide && L <= 8u) {
            bit_transpose<8>(a.w);
#pragma unroll
            for (int k = 0; k < 8; ++k)
                if ((uint32_t)k < L) dst[sgn * (1 + k)] = a.w[k];
        } else {
            bit_transpose<16>(h.w);
#pragma unroll
            for (int k = 0; k < 16; ++k)
                if ((uint32_t)k < L) dst[sgn * (1 + k)] = h.w[k];
        }
    }
    if (block_in_tile < lbytes) {
        const uint32_t wi = 1u + (block_in_tile >> 2);
        reinterpret_cast<unsigned char*>(blob + (sgn > 0 ? org + wi : org - wi))[block_in_tile & 3u] = (unsigned char)L;
    }
    cy.pay_used += round_total;
    cy.wide = __any_sync(kFull, L > 8u);
    return 0;
}

// ---- general route: any code length, any alignment, codes up to 2^30, blobs of any size; straight from and to
// global memory, integer conversion (the definition itself).  Compact rather than fast.

// Sign word and planes of block `bi` of a tile (len elements at xt) into out[0 .. 32] (out[0] = sign word, out[1 + k]
// = plane k); returns the code length.  Positions beyond the tile's end repeat its last element.
__device__ __noinline__ uint32_t general_block(const float* __restrict__ xt, uint32_t bi, uint32_t len, float r, uint32_t* out, float* tmax)
{
    const uint32_t last = len - 1;
    const uint32_t e0 = 32u * bi;
    const uint32_t ep = e0 ? e0 - 1u : 0u;
    const float tp = __fmul_rn(__ldg(xt + (ep < last ? ep : last)), r);
    float tm = fmaxf(*tmax, fabsf(tp));
    uint32_t qp = (uint32_t)__float2int_rn(tp);
    uint32_t m[32];
    uint32_t sg = 0, ob = 0;
#pragma unroll
    for (int j = 0; j < 32; ++j) {
        const uint32_t e = e0 + (uint32_t)j;
        const float t = __fmul_rn(__ldg(xt + (e < last ? e : last)), r);
        tm = fmaxf(tm, fabsf(t));
        const uint32_t q = (uint32_t)__float2int_rn(t);
        const int32_t dd = (int32_t)(q - qp);
        qp = q;
        const uint32_t sm = (uint32_t)(dd >> 31);
        m[j] = (((uint32_t)dd ^ sm) - sm) & 0x7FFFFFFFu;   // |delta|; the mask only matters after a range error
        ob |= m[j];
        sg = __funnelshift_l((uint32_t)dd, sg, 1);
    }
    *tmax = tm;
    bit_transpose<32>(m);
    out[0] = __brev(sg);
#pragma unroll
    for (int k = 0; k < 32; ++k) out[1 + k] = m[k];
    return code_length(ob);
}

// ------------------------------------------------------------------------------------------------ placement

// Position of a tile in its stream = sum of the sizes of the tiles of its job in front of it.  Sizes are published as
// 8-byte states {launch counter, flag, words}, validated by the launch counter instead of being cleared.  Two levels,
// so that a position costs one round trip to L2 even when thousands of tiles finish together (the first wave of a
// launch): tiles of a job form groups of 32;
//   * a tile sums the states of the tiles of its own group in front of it (one window: lane l looks at tile - 1 - l);
//   * the last tile of a group adds its own size and publishes the group's size; when its own position is known it
//     publishes the group's inclusive prefix as well;
//   * the groups in front are summed by a decoupled look-back over the group states (windows of 32 groups = 1024
//     tiles), ending at the first one that carries an inclusive prefix or at the job's first group.
// The search is resumable: a warp that has another tile to encode issues one trip's loads before a round and looks
// at them after it, so the round trip costs it nothing.  Every wait is bounded.
struct LookBack {
    uint32_t ticket, total;     // the tile being placed and its size
    uint32_t first;             // first tile of its group (launch numbering)
    uint32_t gslot0;            // slot of the state of the job's first group
    uint32_t g;                 // the tile's group within the job
    uint32_t grel;              // groups of the job in front of it that are not summed yet
    uint32_t sum_a, sum_b;      // sizes of the tiles of its group in front of it; of the groups summed so far
    bool a_done, b_done, closes_group;
};
__device__ __forceinline__ bool look_back_done(const LookBack& lb) { return lb.a_done && lb.b_done; }
__device__ __forceinline__ uint32_t look_back_result(const LookBack& lb) { return lb.sum_a + lb.sum_b; }

// job_index, tile_begin, tiles_in_job: the tile's job
__device__ __forceinline__ void look_back_begin(LookBack& lb, uint32_t ticket, uint32_t total, int job_index, uint32_t tile_begin,
                                                uint32_t tiles_in_job)
{
    const uint32_t tile = ticket - tile_begin;
    lb.ticket = ticket; lb.total = total;
    lb.g = tile >> 5;
    lb.first = tile_begin + (lb.g << 5);
    lb.gslot0 = (tile_begin >> 5) + (uint32_t)job_index;
    lb.grel = lb.g;
    lb.sum_a = 0; lb.sum_b = 0;
    lb.a_done = (tile & 31u) == 0;
    lb.b_done = lb.g == 0;
    lb.closes_group = (tile & 31u) == 31u || tile + 1 == tiles_in_job;
}

// A tile's size, published as soon as it is known.
__device__ __forceinline__ void publish_size(const Workspace& ws, uint32_t ticket, uint32_t total, uint32_t epoch, int lane)
{
    if (lane == 0 && ticket != ws.skip_publish) st_state(ws.tile_state + ticket, pack_state(epoch, 0u, total));
}

// What the search publishes as it goes, by the tile that closes a group: the group's size once the tiles in front
// are summed, the group's inclusive prefix once the position is known.
__device__ __forceinline__ void look_back_publish(const Workspace& ws, const LookBack& lb, bool a_was_done, uint32_t epoch, int lane)
{
    if (!lb.closes_group || lane != 0 || lb.ticket == ws.skip_publish) return;
    if (look_back_done(lb)) st_state(ws.group_state + lb.gslot0 + lb.g, pack_state(epoch, 1u, lb.sum_a + lb.sum_b + lb.total));
    else if (lb.a_done && !a_was_done) st_state(ws.group_state + lb.gslot0 + lb.g, pack_state(epoch, 0u, lb.sum_a + lb.total));
}

// One trip: NW windows of group states plus the window of the own group, issued together.
template <int NW>
struct LookBackTrip {
    unsigned long long tile_st;
    unsigned long long group_st[NW];
};
template <int NW>
__device__ __forceinline__ void look_back_issue(const Workspace& ws, const LookBack& lb, uint32_t epoch, int lane, LookBackTrip<NW>& tr)
{
    const int at = (int)(lb.ticket - lb.first) - 1 - lane;   // a tile of the own group, counted from the group's first
    tr.tile_st = (!lb.a_done && at >= 0) ? ld_state(ws.tile_state + lb.first + (uint32_t)at) : pack_state(epoch, 0u, 0u);
#pragma unroll
    for (int w = 0; w < NW; ++w) {
        const int gi = (int)lb.grel - 1 - lane - 32 * w;     // a group of the job
        tr.group_st[w] = (!lb.b_done && gi >= 0) ? ld_state(ws.group_state + lb.gslot0 + (uint32_t)gi) : pack_state(epoch, 1u, 0u);
    }
}
// true: progress was made or nothing was left to do (false: a state in the way is not published yet)
template <int NW>
__device__ __forceinline__ bool look_back_eval(const Workspace& ws, LookBack& lb, uint32_t epoch, int lane, const LookBackTrip<NW>& tr)
{
    const bool a_was_done = lb.a_done, was_done = look_back_done(lb);
    bool stuck = false;
    if (!lb.a_done) {
        const bool ready = (uint32_t)(tr.tile_st >> 33) == epoch;   // lanes beyond the group's first tile hold a ready zero
        if (__any_sync(kFull, !ready)) stuck = true;
        else {
            lb.sum_a = __reduce_add_sync(kFull, (uint32_t)tr.tile_st);
            lb.a_done = true;
        }
    }
    bool b_stuck = false;
#pragma unroll
    for (int w = 0; w < NW; ++w) {
        if (!lb.b_done && !b_stuck) {
            const unsigned long long st = tr.group_st[w];
            const bool ready = (uint32_t)(st >> 33) == epoch;
            const unsigned not_ready = __ballot_sync(kFull, !ready);
            const unsigned incl = __ballot_sync(kFull, ready && ((st >> 32) & 1ull));
            const unsigned low = incl & (0u - incl);
            const unsigned upto = incl ? (low | (low - 1u)) : kFull;   // lanes up to the first inclusive one
            if (not_ready & upto) b_stuck = true;
            else {
                lb.sum_b += __reduce_add_sync(kFull, ((upto >> lane) & 1u) ? (uint32_t)st : 0u);
                if (incl) lb.b_done = true;
                else lb.grel -= 32;
            }
        }
    }
    if (!was_done) look_back_publish(ws, lb, a_was_done, epoch, lane);
    return !(stuck || b_stuck);
}
// Runs the search to its end.  false: a state was not published within the poll limit (the time-out is recorded;
// nothing may be written for this tile).
constexpr int kGroupWindows = 2;   // windows of group states per trip of the blocking search
__device__ __forceinline__ bool look_back_finish(const Workspace& ws, LookBack& lb, uint32_t epoch, int lane, uint32_t& status)
{
    int budget = kSpinLimit >> 4;
    uint32_t sleep_ns = 100;   // backs off: polling warps take issue slots from working ones
    while (!look_back_done(lb)) {
        LookBackTrip<kGroupWindows> tr;
        look_back_issue(ws, lb, epoch, lane, tr);
        if (!look_back_eval(ws, lb, epoch, lane, tr)) {
            if (--budget == 0) { status |= kStTimeout; return false; }
            __nanosleep(sleep_ns);
            if (sleep_ns < 1600u) sleep_ns *= 2u;
        }
    }
    return true;
}

__device__ __forceinline__ bool place_tile(const Workspace& ws, uint32_t ticket, int job_index, uint32_t tile_begin, uint32_t tiles_in_job,
                                           uint32_t total, uint32_t epoch, int lane, uint32_t& excl, uint32_t& status)
{
    publish_size(ws, ticket, total, epoch, lane);
    LookBack lb;
    look_back_begin(lb, ticket, total, job_index, tile_begin, tiles_in_job);
    if (look_back_done(lb)) look_back_publish(ws, lb, true, epoch, lane);   // a group of one tile at the job's start
    const bool ok = look_back_finish(ws, lb, epoch, lane, status);
    excl = look_back_result(lb);
    return ok;
}

// Moves a finished blob from the warp's shared memory (word i at blob[org + sgn * i]) to its place in the stream and
// writes what goes with it: index entry, stream length (last tile), header (first tile).
__device__ __forceinline__ void emit_tile(const Job& job, uint32_t tile, const uint32_t* __restrict__ blob, uint32_t org, int sgn,
                                          uint32_t total, uint32_t excl, bool placed, float eb_abs, float s, int lane, uint32_t& status)
{
    const uint32_t nT = (uint32_t)((job.n + kTile - 1) / kTile);
    const unsigned long long word0 = (unsigned long long)kHeaderWords + nT + excl;
    const bool fits = (word0 + total) * 4ull <= job.out_cap;
    if (!fits) status |= kStCapacity;
    const bool go = fits && placed;
    if (go) {
        uint32_t* __restrict__ dst = job.out + word0;
        const uint32_t* src = blob + org + sgn * lane;
        const int step = 32 * sgn;
#pragma unroll 4
        for (uint32_t i = lane; i < total; i += 32, src += step) dst[i] = *src;
    }
    if (lane == 0) {
        if (go) job.out[kHeaderWords + tile] = excl + total;
        if (tile == nT - 1) *job.out_bytes = (size_t)((word0 + total) * 4ull);
    }
    if (tile == 0) write_header(job.out, lane, job.n, eb_abs, s, nT);
}

// A tile whose blob sits in the warp's shared memory, size published, position being looked for.
struct PendingTile {
    bool valid;
    int job;
    uint32_t dir;
    LookBack lb;
};

// Completes the search for the waiting tile's position and moves the tile to the stream.
__device__ __noinline__ uint32_t flush_tile(const JobBatch* jb, Workspace ws, int job, uint32_t dir, LookBack lb, const uint32_t* blob,
                                            uint32_t blob_words, uint32_t epoch, float eb_abs, float s, int lane)
{
    const Job& jp = jb->job[job];
    uint32_t st = 0;
    const bool placed = look_back_finish(ws, lb, epoch, lane, st);
    emit_tile(jp, lb.ticket - jp.tile_begin, blob, dir ? blob_words - 1u : 0u, dir ? -1 : 1, lb.total, look_back_result(lb), placed, eb_abs,
              s, lane, st);
    return st;
}

__device__ __forceinline__ uint32_t take_ticket(const Workspace& ws, int lane)
{
    uint32_t t = 0;
    if (lane == 0) t = atomicAdd(ws.ticket, 1u);
    return __shfl_sync(kFull, t, 0);
}

// ------------------------------------------------------------------------------------------------ compress

// Encodes one tile by the general route: the sizes of all its blocks first, then its placement, then every block once
// more, written straight into the stream.
__device__ __noinline__ uint32_t encode_tile_general(const float* __restrict__ x, uint32_t* __restrict__ out, size_t* out_bytes,
                                                     unsigned long long n, unsigned long long out_cap, int job_index, uint32_t tile_begin,
                                                     uint32_t ticket, float r, float s, float eb_abs, Workspace ws, uint32_t epoch, int lane)
{
    uint32_t status = 0;
    const uint32_t tile = ticket - tile_begin;
    const unsigned long long start = (unsigned long long)tile * kTile;
    const uint32_t nT = (uint32_t)((n + kTile - 1) / kTile);
    const uint32_t len = (uint32_t)((n - start < (unsigned long long)kTile) ? (n - start) : kTile);
    const uint32_t nb = (len + kBlock - 1) / kBlock;
    const uint32_t padw = (nb + 3) >> 2;
    const float* __restrict__ xt = x + start;
    uint32_t planes[33];
    float tmax = 0.0f;
    uint32_t lens = 0;      // byte rd: code length of block 32 rd + lane
    uint32_t offs[kRoundsPerTile];
    uint32_t used = 0;
#pragma unroll
    for (int rd = 0; rd < kRoundsPerTile; ++rd) {
        const uint32_t bi = 32u * rd + (uint32_t)lane;
        uint32_t L = 0;
        if (bi < nb) L = general_block(xt, bi, len, r, planes, &tmax);
        const uint32_t nw = L ? L + 1u : 0u;
        const uint32_t incl = warp_incl_scan(nw, lane);
        offs[rd] = used + incl - nw;
        used += __shfl_sync(kFull, incl, 31);
        lens |= L << (8 * rd);
    }
    if (!(tmax < 1073741824.0f)) status |= kStRange;
    else if (tmax > 32768.5f) status |= kStPrecision;
    const uint32_t total = 1u + padw + used;
    uint32_t excl = 0;
    const bool placed = place_tile(ws, ticket, job_index, tile_begin, nT, total, epoch, lane, excl, status);
    const unsigned long long word0 = (unsigned long long)kHeaderWords + nT + excl;
    const bool fits = (word0 + total) * 4ull <= out_cap;
    if (!fits) status |= kStCapacity;
    const bool go = fits && placed;
    if (go) {
        uint32_t* __restrict__ dst = out + word0;
#pragma unroll
        for (int rd = 0; rd < kRoundsPerTile; ++rd) {
            const uint32_t bi = 32u * rd + (uint32_t)lane;
            const uint32_t L = (lens >> (8 * rd)) & 0xFFu;
            if (bi < 4u * padw) reinterpret_cast<unsigned char*>(dst + 1)[bi] = (unsigned char)L;
            if (L) {
                float unused = 0.0f;
                (void)general_block(xt, bi, len, r, planes, &unused);
                uint32_t* d = dst + 1 + padw + offs[rd];
                for (uint32_t k = 0; k <= L; ++k) d[k] = planes[k];
            }
        }
        if (lane == 0) {
            dst[0] = (uint32_t)__float2int_rn(__fmul_rn(__ldg(xt), r));
            out[kHeaderWords + tile] = excl + total;
        }
    }
    if (lane == 0 && tile == nT - 1) *out_bytes = (size_t)((word0 + total) * 4ull);
    if (tile == 0) write_header(out, lane, n, eb_abs, s, nT);
    return status;
}

// A warp's blob area holds two tiles: the one being encoded and the one before it, which waits there for its
// placement until the warp has encoded the next one (by then the tiles in front of it have published their sizes, so
// the look-back does not wait).  The two share the area from its two ends: one blob grows upwards from word 0, the
// other downwards from the last word, alternating, so that only their sum is limited.
constexpr int kEncBlobWords = 1536;
struct EncWarpShared {
    alignas(16) float stage[2][kRound];
    alignas(16) uint32_t blob[kEncBlobWords];
};

// A tile of the launch as a warp sees it.
struct TileInfo {
    int job;            // -1: beyond the launch's last tile
    uint32_t tile;      // number within the job
    uint32_t tiles;     // tiles of the job
    uint32_t len;       // elements (0: a job without elements, or no valid bound: header and length only)
    const float* xt;    // the tile's first element
};

__global__ void __launch_bounds__(kCodecThreads, 16 / kCodecWarps) enc_kernel(const __grid_constant__ JobBatch jb, Workspace ws, Params hp, int use_dev_params)
{
    pdl_enter();
    extern __shared__ __align__(16) unsigned char smem_raw[];
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    EncWarpShared& sh = reinterpret_cast<EncWarpShared*>(smem_raw)[warp];
    const uint32_t epoch = *reinterpret_cast<volatile uint32_t*>(ws.epoch);
    uint32_t status = 0;
    Params prm = hp;
    if (use_dev_params) prm = *ws.params;
    const float r = prm.r, s = prm.s, eb_abs = prm.eb_abs;
    const uint32_t rl = (uint32_t)lane >> 3, lc = (uint32_t)lane & 7u;
    const uint32_t lane_off0 = rl * 128u + ((lc ^ rl) << 4), lane_off1 = rl * 128u + ((lc ^ (rl | 4u)) << 4);

    // the job of the tile looked up last: consecutive look-ups mostly stay inside it
    int cj = -1;
    uint32_t cj_begin = 0, cj_count = 0;
    const float* cj_x = nullptr;
    unsigned long long cj_n = 0;
    auto locate = [&](uint32_t t) {
        TileInfo ti;
        ti.job = -1; ti.tile = 0; ti.tiles = 1; ti.len = 0; ti.xt = nullptr;
        if (t >= jb.total_tiles) return ti;
        if (t - cj_begin >= cj_count) {
            cj = find_job(jb, t);
            const Job& q = jb.job[cj];
            cj_begin = q.tile_begin;
            cj_count = (cj + 1 < jb.count ? jb.job[cj + 1].tile_begin : jb.total_tiles) - cj_begin;
            cj_x = q.x;
            cj_n = q.n;
        }
        ti.job = cj;
        ti.tile = t - cj_begin;
        ti.tiles = cj_count;
        const unsigned long long start = (unsigned long long)ti.tile * kTile;
        if (cj_n && prm.valid) {
            ti.len = (uint32_t)((cj_n - start < (unsigned long long)kTile) ? (cj_n - start) : kTile);
            ti.xt = cj_x + start;
        }
        return ti;
    };

    PendingTile pend;
    pend.valid = false; pend.job = 0; pend.dir = 1;
    look_back_begin(pend.lb, 0, 0, 0, 0, 1);
    auto flush_pending = [&]() {
        status |= flush_tile(&jb, ws, pend.job, pend.dir, pend.lb, sh.blob, kEncBlobWords, epoch, eb_abs, s, lane);
        __syncwarp();   // the waiting tile's end of the blob area is free once every lane has read its share
        pend.valid = false;
    };

    TR_DECL;
#ifdef ZCCL_TRACE
    unsigned long long tr_tile_end[3] = {0, 0, 0}; unsigned tr_ntiles = 0;
#endif
    uint32_t ticket = take_ticket(ws, lane);
#ifdef ZCCL_TRACE
    const unsigned tr_first_ticket = ticket;
#endif
    TileInfo cur = locate(ticket);
    uint32_t p = 0;   // stage that holds (or will hold) the round about to be encoded
    if (cur.len) load_round(sh.stage[p], cur.xt, 0, cur.len, lane, lane_off0, lane_off1);
    cp_async_commit();

    while (cur.job >= 0) {
        const uint32_t tile_begin = ticket - cur.tile;
        const uint32_t len = cur.len;
        const uint32_t nb = (len + kBlock - 1) / kBlock;
        const uint32_t padw = (nb + 3) >> 2;
        const uint32_t rounds = (nb + 31) >> 5;
        const float* __restrict__ xt = cur.xt;
        const uint32_t dir = pend.dir ^ 1u;   // the end of the blob area the waiting tile does not use
        const uint32_t org = dir ? (uint32_t)kEncBlobWords - 1u : 0u;
        const int sgn = dir ? -1 : 1;

        // the number of the tile after this one is asked for now and looked at in the last round
        uint32_t next_raw = 0;
        if (lane == 0) next_raw = atomicAdd(ws.ticket, 1u);
        uint32_t next = 0;
        TileInfo nxt;
        nxt.job = -1; nxt.tile = 0; nxt.tiles = 1; nxt.len = 0; nxt.xt = nullptr;

        EncodeCarry cy;
        cy.pay_used = 0; cy.wide = false;
        float carry_x = 0.0f;
        int32_t q_first = 0;
        bool general = false;
        TR_MARK(0);   // tile set-up
        // a tile without elements runs the loop once, for the hand-over to the next tile only
        for (uint32_t rd = 0; rd < (rounds ? rounds : 1u); ++rd) {
            __syncwarp();   // every lane is done with the other stage (it held the round before this one)
            const bool last_round = rd + 1 >= rounds;
            if (last_round) {
                next = __shfl_sync(kFull, next_raw, 0);
                nxt = locate(next);
                if (nxt.len) load_round(sh.stage[p ^ 1u], nxt.xt, 0, nxt.len, lane, lane_off0, lane_off1);
            } else {
                load_round(sh.stage[p ^ 1u], xt, (rd + 1) * kRound, len, lane, lane_off0, lane_off1);
            }
            cp_async_commit();
            if (rounds == 0) { cp_async_wait<1>(); break; }
            // one window of the waiting tile's look-back rides along with this round
            const bool looking = pend.valid && !look_back_done(pend.lb);
            LookBackTrip<1> trip;
            if (looking) look_back_issue(ws, pend.lb, epoch, lane, trip);
            TR_MARK(1);   // request of the next round
            cp_async_wait<1>();
            __syncwarp();   // the round's copies of all lanes have landed
            TR_MARK(2);   // wait for this round's data
            const float* st = sh.stage[p];
            const char* row = reinterpret_cast<const char*>(st) + 128 * lane;
            const uint32_t sw = ((uint32_t)lane & 7u) << 4;
            float xprev = lane ? read_last_of_row(st, (uint32_t)lane - 1u) : carry_x;
            if (rd == 0 && lane == 0) {
                xprev = *reinterpret_cast<const float*>(row);   // the tile's first element is its own predecessor
                // exact while |x r| < 2^22; a larger first code sends the tile to the general route anyway
                q_first = (int32_t)(__float_as_uint(__fadd_rn(__fmul_rn(xprev, r), kRoundMagic)) - kRoundMagicBits);
            }
            carry_x = read_last_of_row(st, 31);
            const uint32_t bi = 32u * rd + (uint32_t)lane;
            const uint32_t room = (uint32_t)kEncBlobWords - 1u - padw;
            int rc;
            for (;;) {
                const uint32_t held = pend.valid ? pend.lb.total : 0u;
                rc = encode_round(row, sw, xprev, r, bi < nb, bi, 4u * padw, sh.blob, org, sgn, 1u + padw, room > held ? room - held : 0u, cy,
                                  lane, status);
                if (rc != 2 || !pend.valid) break;
                flush_pending();   // no room next to the waiting tile: place that one now, then try again
            }
            TR_MARK(3);   // encode
            if (looking && pend.valid) (void)look_back_eval(ws, pend.lb, epoch, lane, trip);
            TR_MARK(4);   // look-back evaluation
            p ^= 1u;
            if (rc != 0) {
                general = true;
                if (!last_round) {   // hand over to the next tile: its first round goes where this tile's next round was asked into
                    cp_async_wait<0>();
                    __syncwarp();
                    next = __shfl_sync(kFull, next_raw, 0);
                    nxt = locate(next);
                    if (nxt.len) load_round(sh.stage[p], nxt.xt, 0, nxt.len, lane, lane_off0, lane_off1);
                    cp_async_commit();
                }
                break;
            }
        }
        if (len == 0) {
            const Job& job = jb.job[cur.job];
            const bool hdr = prm.valid && job.out_cap >= (unsigned)kHeaderBytes;
            if (lane == 0) {
                st_state(ws.tile_state + ticket, pack_state(epoch, 0u, 0u));
                if (cur.tile == 0) *job.out_bytes = hdr ? kHeaderBytes : 0;
            }
            if (hdr && cur.tile == 0) write_header(job.out, lane, 0, eb_abs, s, 0);
            p ^= 1u;
        } else if (general) {
            const Job& job = jb.job[cur.job];
            status |= encode_tile_general(job.x, job.out, job.out_bytes, job.n, job.out_cap, cur.job, tile_begin, ticket, r, s, eb_abs, ws, epoch,
                                          lane);
        } else {
            if (lane == 0) sh.blob[org] = (uint32_t)q_first;
            const uint32_t total = 1u + padw + cy.pay_used;
            publish_size(ws, ticket, total, epoch, lane);
            __syncwarp();   // the blob's words, written by all lanes, are visible to all
            TR_MARK(5);   // publish
#ifdef ZCCL_TRACE
            if (tr_ntiles < 3) tr_tile_end[tr_ntiles] = gtime();
            ++tr_ntiles;
#endif
            if (pend.valid) flush_pending();
            pend.valid = true; pend.job = cur.job; pend.dir = dir;
            look_back_begin(pend.lb, ticket, total, cur.job, tile_begin, cur.tiles);
            if (look_back_done(pend.lb)) look_back_publish(ws, pend.lb, true, epoch, lane);   // a group of one tile at the job's start
            TR_MARK(6);   // flush of the waiting tile
        }
        cur = nxt;
        ticket = next;
    }
    if (pend.valid) flush_pending();
    TR_MARK(7);   // last flush
    TR_FLUSH;
#ifdef ZCCL_TRACE
    if (lane == 0) { unsigned long long* rec = g_rec + 8 * (blockIdx.x * kCodecWarps + warp); rec[0] = tr_g0; rec[1] = tr_tile_end[0]; rec[2] = tr_tile_end[1]; rec[3] = tr_tile_end[2]; rec[4] = gtime(); rec[5] = tr_ntiles; rec[6] = tr_first_ticket; }
#endif
    cp_async_wait<0>();
    if (status) atomicOr(ws.status, status);
    finish_launch(ws, epoch, tid, ws.ticket);
}

// Per-device launch set-up (shared-memory attribute, resident CTAs per SM), done once per device under a lock.
constexpr int kMaxDevices = 64;
struct DeviceSetup {
    bool ready = false;
    int enc_ctas = 1;
};
DeviceSetup g_dev[kMaxDevices];
std::mutex g_dev_mu;

cudaError_t device_setup(const DeviceSetup** out)
{
    int dev = 0;
    cudaError_t e = cudaGetDevice(&dev);
    if (e != cudaSuccess) return e;
    if (dev < 0 || dev >= kMaxDevices) return cudaErrorInvalidDevice;
    std::lock_guard<std::mutex> lock(g_dev_mu);
    DeviceSetup& d = g_dev[dev];
    if (!d.ready) {
        e = cudaFuncSetAttribute(enc_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)(sizeof(EncWarpShared) * kCodecWarps));
        if (e != cudaSuccess) return e;
        int a = 0;
        e = cudaOccupancyMaxActiveBlocksPerMultiprocessor(&a, enc_kernel, kCodecThreads, sizeof(EncWarpShared) * kCodecWarps);
        if (e != cudaSuccess) return e;
        d.enc_ctas = a > 0 ? a : 1;
        d.ready = true;
    }
    *out = &d;
    return cudaSuccess;
}

}  // namespace

#ifdef ZCCL_TRACE
extern "C" int zccl_debug_rec(unsigned long long* out, int n) { return cudaMemcpyFromSymbol(out, g_rec, sizeof(unsigned long long) * n) == cudaSuccess ? 0 : -1; }
extern "C" int zccl_debug_trace(unsigned long long* out16)
{
    unsigned long long z[16] = {};
    z[9] = z[11] = ~0ull;
    if (cudaMemcpyFromSymbol(out16, g_trace, sizeof(z)) != cudaSuccess) return -1;
    return cudaMemcpyToSymbol(g_trace, z, sizeof(z)) == cudaSuccess ? 0 : -1;
}
#endif

cudaError_t launch_encode_lanes(const JobBatch& jb, const Workspace& ws, bool device_params, Params host_params, int sm_count,
                                cudaStream_t st)
{
    const DeviceSetup* d = nullptr;
    cudaError_t e = device_setup(&d);
    if (e != cudaSuccess) return e;
    const unsigned long long want = ((unsigned long long)jb.total_tiles + kCodecWarps - 1) / kCodecWarps;
    unsigned long long cap = (unsigned long long)sm_count * d->enc_ctas;
#ifdef ZCCL_TRACE
    if (const char* e = getenv("ZCCL_EXP_CTAS")) cap = (unsigned long long)sm_count * atoi(e);
#endif
    const unsigned grid = (unsigned)(want < cap ? want : cap);
    return launch_k(enc_kernel, dim3(grid), dim3(kCodecThreads), sizeof(EncWarpShared) * kCodecWarps, st, jb, ws, host_params,
                    device_params ? 1 : 0);
}

}  // namespace zccl
