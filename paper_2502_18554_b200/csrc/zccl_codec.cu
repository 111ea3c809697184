// fZ-light codec kernels for sm_100a: encoder, decoder and the fused decode + reduce + encode hop.
//
// Work decomposition: ONE LANE OWNS ONE 32-ELEMENT BLOCK.  A warp works on a round of 32 blocks (1024 elements,
// a quarter of a tile); lane l holds the 32 consecutive elements of block l in registers.  Everything the format
// asks of a block then happens inside one thread, with no shuffle, vote or barrier:
//   * quantise and 1-D Lorenzo delta: fp32 on the FMA pipe (t + 1.5 * 2^23 rounds to nearest even, deltas of two
//     such values are exact, |delta| + 2^23 has the magnitude in its mantissa);
//   * code length: OR of the 32 magnitudes, one count-leading-zeros;
//   * bit planes: the magnitudes are packed four (code lengths up to 8), two (up to 16) or one to a word by byte
//     permutes and an in-register bit-matrix transpose (3, 4 or 5 stages of shift + bit-select pairs) turns them
//     into plane words; the decoder runs the same transpose backwards and gets the block's delta sum from
//     population counts of the planes;
//   * sign word: one funnel shift per element.
// A warp needs its neighbours only for the prefix sum of the blocks' sizes and, when it decodes, of the blocks'
// delta sums (one shuffle scan per round each).  Warps never wait for each other: there is no __syncthreads and no
// inter-CTA wait in the round loops.  The loops over a block's elements are rolled on purpose: the unrolled forms
// were bound by instruction fetch.
//
// Memory.  A lane wants 128 consecutive bytes per block while global accesses must be contiguous across the warp,
// so rounds go through shared memory.  The array is described to the copy engine as rows of 32 floats (one tensor
// map per chunk-operation, built on the host); one tiled tensor copy brings a round's 32 rows into a 4 KiB stage
// in the 128-byte swizzle (16-byte chunk c of row t at c ^ (t & 7)), one round ahead, completion on an mbarrier;
// the lanes' 128-bit row reads and (decoder) row writes are free of bank conflicts; decoded rounds leave by a
// tensor store.  Ragged or misaligned rounds take plain loads and stores into the same layout.  Compressed bytes
// move with untiled bulk copies.
//
// Compression takes two launches and no waits:
//   1. encode_rounds_kernel: rounds are dealt round-robin to the warps of the grid; each is encoded into a fixed
//      slot of the workspace (code-length bytes, then the payload), its payload size recorded, and added to the
//      sum of its group of 32 tiles;
//   2. place_kernel: one CTA per group turns the group sums in front of it and its own rounds' sizes into stream
//      positions, writes index entries, outliers and code lengths and moves the payloads from the slots.
// The fused hop (hop_tiles_kernel) is the same first step with a decoder in front: the incoming round is decoded
// in place onto the stage that holds the local operand, reduced, optionally stored, and re-encoded from the stage.
// The slots cost a write and a read of the compressed bytes, mostly absorbed by L2; in exchange no warp ever waits
// for another, so nothing depends on which CTAs are resident together.
//
// A single-pass encoder (enc_kernel: a warp per tile, positions by a two-level decoupled look-back over per-tile and
// per-group states, every wait bounded and reported through the status word) remains for contexts without slots:
// the allocation-free entry point.
//
// Binary64 input has kernels of the same design with 8 KiB rounds (zccl_codec_f64.cuh, included below; they share
// the back ends, the slots and place_kernel).
#include "zccl_device.cuh"

#include <cuda.h>
#include <cstring>
#include <mutex>

namespace zccl {
namespace {

constexpr int kCodecWarps = 4;                        // warps per CTA, each with tiles of its own
constexpr int kCodecThreads = 32 * kCodecWarps;
constexpr int kRound = 32 * kBlock;                   // elements per round: one block per lane
constexpr int kRoundsPerTile = kTile / kRound;
constexpr int kLWords = kBlocksPerTile / 4;           // code-length words of a full tile

// ------------------------------------------------------------------------------------------------ small pieces

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
// (The stages are separate instantiations rather than a loop over d: left to the unroller, the 16-word form kept its
// words in local memory, indexed at run time.)
template <int N, int D>
__device__ __forceinline__ void bit_transpose_stage(uint32_t (&w)[N])
{
    constexpr uint32_t m = D == 16 ? 0x0000FFFFu : D == 8 ? 0x00FF00FFu : D == 4 ? 0x0F0F0F0Fu : D == 2 ? 0x33333333u : 0x55555555u;
#pragma unroll
    for (int i = 0; i < N; ++i) {
        if (i & D) continue;
        const uint32_t a = w[i], b = w[i + D];
        w[i] = (a & m) | ((b << D) & ~m);
        w[i + D] = ((a >> D) & m) | (b & ~m);
    }
}
template <int N>
__device__ __forceinline__ void bit_transpose(uint32_t (&w)[N])
{
    if constexpr (N >= 32) bit_transpose_stage<N, 16>(w);
    if constexpr (N >= 16) bit_transpose_stage<N, 8>(w);
    bit_transpose_stage<N, 4>(w);
    bit_transpose_stage<N, 2>(w);
    bit_transpose_stage<N, 1>(w);
}

// ------------------------------------------------------------------------------------------------ stages

// A stage holds one round: row t = the 32 floats of block t (128 bytes), its 16-byte chunk c stored at chunk
// position c ^ (t & 7) of the row, so that the lanes' 128-bit reads of their own rows fall into different banks.
// That is the 128-byte swizzle of the tensor copy engine: a full round of an array that starts on a 16-byte boundary
// is brought in by ONE tiled tensor copy (32 rows x 32 floats of the array seen as rows of 32 floats; issued by one
// lane, completion on the stage's mbarrier).  Besides costing no instructions, this keeps the load/store path free:
// with the input streamed through it (16-byte asynchronous copies were tried first), every latency-critical load
// of the placement (the states of other tiles) queued up behind kilobytes of input and took microseconds.  Stages
// must start on a 1024-byte boundary (the swizzle works on address bits).  Other rounds (ragged ends, unaligned
// arrays) are loaded element by element, positions beyond the tile's end repeating its last element (so that the
// padding of the last block has zero deltas).
__device__ __forceinline__ uint32_t stage_chunk_byte(uint32_t row, uint32_t chunk) { return row * 128u + ((chunk ^ (row & 7u)) << 4); }

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
// Tiled tensor copy of rows [row0, row0 + 32) of the array behind `map` into a stage (one thread).
__device__ __forceinline__ void tensor_load_round(float* stage, unsigned long long* bar, const CUtensorMap* map, uint32_t row0)
{
    mbar_expect_tx(bar, kRound * 4);
    asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
    asm volatile("cp.async.bulk.tensor.2d.shared::cluster.global.tile.mbarrier::complete_tx::bytes [%0], [%1, {%2, %3}], [%4];"
                 ::"r"(smem_u32(stage)), "l"(map), "r"(0), "r"((int)row0), "r"(smem_u32(bar)) : "memory");
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
    // the multiplications, the additions of the rounding constant and the guard's sums go two elements to an instruction
    // (sm_100's packed fp32: each half rounds as the scalar operation does; 23.3 -> 23.0 us per 64 MiB)
    float2 acc2 = make_float2(__fmul_rn(tp, tp), 0.0f);
    const float2 r2 = make_float2(r, r), magic2 = make_float2(kRoundMagic, kRoundMagic);
    uint32_t orb = 0, sg = 0;
#pragma unroll
    for (int i = 0; i < N; ++i) o.w[i] = 0;
#pragma unroll 1
    for (uint32_t g = 0; g < 32u / N; ++g) {
#pragma unroll
        for (int q = 0; q < N / 4; ++q) {
            const float4 v = *reinterpret_cast<const float4*>(row + ((16u * (g * (N / 4) + q)) ^ sw));
            const float2 t01 = __fmul2_rn(make_float2(v.x, v.y), r2), t23 = __fmul2_rn(make_float2(v.z, v.w), r2);
            acc2 = __ffma2_rn(t01, t01, acc2);
            acc2 = __ffma2_rn(t23, t23, acc2);
            // (the products are used twice, by the guard and here; the compiler was seen to contract a packed product with
            // ONE use and the packed addition behind it into a packed fused multiply-add whatever --fmad says, which the
            // full-size parity tests would show as codes that differ at ties)
            const float2 c01 = __fadd2_rn(t01, magic2), c23 = __fadd2_rn(t23, magic2);
            const float cs[4] = {c01.x, c01.y, c23.x, c23.y};
#pragma unroll
            for (int e = 0; e < 4; ++e) {
                const float c = cs[e];
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
    o.guard = __fadd_rn(acc2.x, acc2.y);
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
// outgrow `pay_cap` payload words.  `mid` is called once, by all lanes, when the rows have been read and the sizes are
// known, before anything is stored.
// This is one width class (N = 8 or 16 bits per packed magnitude); it returns 3, with nothing stored and `mid` not
// called, when a lane's code is longer than N.
template <int N, class Mid>
__device__ __forceinline__ int encode_round_n(const char* row, uint32_t sw, float xprev, float r, bool active, uint32_t block_in_tile,
                                              uint32_t lbytes, uint32_t* __restrict__ blob, uint32_t org, int sgn, uint32_t pay_base,
                                              uint32_t pay_cap, EncodeCarry& cy, int lane, uint32_t& status, Mid&& mid)
{
    BlockPack<N> a;
    block_pass<N>(row, sw, xprev, r, a);
    uint32_t L = active ? code_length(a.orb) : 0u;
    if (N == 8 && __any_sync(kFull, L > 8u)) return 3;
    const bool beyond = !(a.guard < kGuardExact) || L > 16u;
    const uint32_t nw = L ? L + 1u : 0u;
    const uint32_t incl = warp_incl_scan(nw, lane);
    const uint32_t round_total = __shfl_sync(kFull, incl, 31);
    mid();   // the caller's business between the two halves (all lanes, once per round)
    if (__any_sync(kFull, beyond)) return 1;
    if (cy.pay_used + round_total > pay_cap) return 2;
    if (a.guard >= kGuardSmall && block_tmax(row, sw, r) > 32768.5f) status |= kStPrecision;
    __syncwarp();   // every lane has read its row for the last time: the blob may lie over the stage
    if (L) {
        uint32_t* dst = blob + ((int)org + sgn * (int)(pay_base + cy.pay_used + (incl - nw)));
        dst[0] = a.sign;
        bit_transpose<N>(a.w);
#pragma unroll
        for (int k = 0; k < N; ++k)
            if ((uint32_t)k < L) dst[sgn * (1 + k)] = a.w[k];
    }
    if (block_in_tile < lbytes) {
        const uint32_t wi = 1u + (block_in_tile >> 2);
        reinterpret_cast<unsigned char*>(blob + (sgn > 0 ? org + wi : org - wi))[block_in_tile & 3u] = (unsigned char)L;
    }
    cy.pay_used += round_total;
    cy.wide = __any_sync(kFull, L > 8u);
    return 0;
}

// One width class for the whole warp: a pass at 8 bits first unless the round before was wide; if any lane then has a
// longer code, every lane repeats the pass at 16 bits (the warp would execute those instructions anyway, and with
// one class at a time only one set of packed words is alive).
template <class Mid>
__device__ __forceinline__ int encode_round(const char* row, uint32_t sw, float xprev, float r, bool active, uint32_t block_in_tile,
                                            uint32_t lbytes, uint32_t* __restrict__ blob, uint32_t org, int sgn, uint32_t pay_base,
                                            uint32_t pay_cap, EncodeCarry& cy, int lane, uint32_t& status, Mid&& mid)
{
    if (!cy.wide) {
        const int rc = encode_round_n<8>(row, sw, xprev, r, active, block_in_tile, lbytes, blob, org, sgn, pay_base, pay_cap, cy, lane, status, mid);
        if (rc != 3) return rc;
    }
    return encode_round_n<16>(row, sw, xprev, r, active, block_in_tile, lbytes, blob, org, sgn, pay_base, pay_cap, cy, lane, status, mid);
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
    uint32_t gsize;             // tiles of that group
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
    lb.gsize = tiles_in_job - (lb.g << 5) < 32u ? tiles_in_job - (lb.g << 5) : 32u;
}

// A tile's size, published as soon as it is known (one thread): its own state, and its share of its group's
// accumulator {tiles:24 | words:40}.  The tile whose addition completes the group publishes the group's size, so a
// group's size never waits for anybody's position.  Split in two, so that the caller can do other work while the
// addition is on its way.
constexpr unsigned long long kAccWordsMask = (1ull << 40) - 1ull;
__device__ __forceinline__ unsigned long long publish_size_issue(const Workspace& ws, const LookBack& lb)
{
    if (lb.ticket == ws.skip_publish) return ~0ull;
    const unsigned long long old = atomicAdd(ws.group_acc + lb.gslot0 + lb.g, (1ull << 40) | (unsigned long long)lb.total);
    return old;
}
__device__ __forceinline__ void publish_size_finish(const Workspace& ws, const LookBack& lb, unsigned long long old, uint32_t epoch)
{
    if (old == ~0ull) return;
    if ((uint32_t)(old >> 40) + 1u == lb.gsize)
        st_state(ws.group_state + lb.gslot0 + lb.g, pack_state(epoch, 0u, (uint32_t)(old & kAccWordsMask) + lb.total));
}
__device__ __forceinline__ void publish_tile_state(const Workspace& ws, uint32_t ticket, uint32_t total, uint32_t epoch)
{
    if (ticket != ws.skip_publish) st_state(ws.tile_state + ticket, pack_state(epoch, 0u, total));
}

// The tile that closes a group publishes the group's inclusive prefix once its own position is known.
__device__ __forceinline__ void look_back_publish(const Workspace& ws, const LookBack& lb, uint32_t epoch, int lane)
{
    if (!lb.closes_group || lane != 0 || lb.ticket == ws.skip_publish || !look_back_done(lb)) return;
    st_state(ws.group_state + lb.gslot0 + lb.g, pack_state(epoch, 1u, lb.sum_a + lb.sum_b + lb.total));
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
    const bool was_done = look_back_done(lb);
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
    if (!was_done) look_back_publish(ws, lb, epoch, lane);
    return !(stuck || b_stuck);
}
// Runs the search to its end.  false: a state was not published within the poll limit (the time-out is recorded;
// nothing may be written for this tile).
constexpr int kGroupWindows = 4;   // windows of group states per trip of the blocking search
__device__ __forceinline__ bool look_back_finish(const Workspace& ws, LookBack& lb, uint32_t epoch, int lane, uint32_t& status)
{
    int budget = kSpinLimit >> 4;
    uint32_t sleep_ns = 0;   // the first polls follow each other at once; then the warp backs off (polling takes issue slots)
    while (!look_back_done(lb)) {
        LookBackTrip<kGroupWindows> tr;
        look_back_issue(ws, lb, epoch, lane, tr);
        if (!look_back_eval(ws, lb, epoch, lane, tr)) {
            if (--budget == 0) { status |= kStTimeout; return false; }
            if (budget < (kSpinLimit >> 4) - 6) {
                sleep_ns = sleep_ns < 400u ? sleep_ns + 100u : 400u;
                __nanosleep(sleep_ns);
            }
        }
    }
    return true;
}

__device__ __forceinline__ bool place_tile(const Workspace& ws, uint32_t ticket, int job_index, uint32_t tile_begin, uint32_t tiles_in_job,
                                           uint32_t total, uint32_t epoch, int lane, uint32_t& excl, uint32_t& status)
{
    LookBack lb;
    look_back_begin(lb, ticket, total, job_index, tile_begin, tiles_in_job);
    if (lane == 0) {
        publish_tile_state(ws, ticket, total, epoch);
        publish_size_finish(ws, lb, publish_size_issue(ws, lb), epoch);
    }
    if (look_back_done(lb)) look_back_publish(ws, lb, epoch, lane);   // the job's first tile
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
constexpr int kEncBlobWords = 2556;
struct alignas(1024) EncWarpShared {
    float stage[2][kRound];                 // each on a 1024-byte boundary
    uint32_t blob[kEncBlobWords];
    alignas(8) unsigned long long bar[2];   // completion of the tensor copies into each stage
};
static_assert(sizeof(EncWarpShared) == 18 * 1024, "a warp's share of the shared memory");

// One tensor map per job of a launch: the job's input seen as rows of 32 floats.
template <int CAP>
struct alignas(64) TileMapsT {
    CUtensorMap m[CAP];
};
using TileMaps = TileMapsT<kMaxJobs>;

// A tile of the launch as a warp sees it.
struct TileInfo {
    int job;            // -1: beyond the launch's last tile
    uint32_t tile;      // number within the job
    uint32_t tiles;     // tiles of the job
    uint32_t len;       // elements (0: a job without elements, or no valid bound: header and length only)
    const float* xt;    // the tile's first element
    bool mapped;        // the job's input has a tensor map (16-byte aligned, at least one row)
};

__global__ void __launch_bounds__(kCodecThreads, 12 / kCodecWarps) enc_kernel(const __grid_constant__ JobBatch jb, const __grid_constant__ TileMaps maps, Workspace ws, Params hp,
                                                                               int use_dev_params)
{
    pdl_enter();
    extern __shared__ __align__(16) unsigned char smem_raw[];
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    EncWarpShared& sh = reinterpret_cast<EncWarpShared*>(smem_raw + ((1024u - (smem_u32(smem_raw) & 1023u)) & 1023u))[warp];
    const uint32_t epoch = *reinterpret_cast<volatile uint32_t*>(ws.epoch);
    uint32_t status = 0;
    Params prm = hp;
    if (use_dev_params) prm = *ws.params;
    const float r = prm.r, s = prm.s, eb_abs = prm.eb_abs;
    if (lane == 0) {
        mbar_init(&sh.bar[0], 1);
        mbar_init(&sh.bar[1], 1);
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    __syncwarp();
    uint32_t fills0 = 0, fills1 = 0;      // bulk rounds completed per stage (phase parity of its mbarrier)
    bool bulk0 = false, bulk1 = false;    // the round on its way into each stage comes by bulk copies
    // asks for the round that starts at element e0 of a tile into stage `buf` (nothing for a tile without elements)
    auto request = [&](uint32_t buf, const TileInfo& ti, uint32_t e0) {
        bool bulk = false;
        if (ti.len) {
            if (ti.mapped && e0 + (uint32_t)kRound <= ti.len) {
                if (lane == 0) tensor_load_round(sh.stage[buf], &sh.bar[buf], &maps.m[ti.job], ti.tile * (uint32_t)kBlocksPerTile + (e0 >> 5));
                bulk = true;
            } else load_round_ragged(sh.stage[buf], ti.xt, e0, ti.len, lane);
        }
        if (buf) bulk1 = bulk; else bulk0 = bulk;
    };
    // waits for the round in stage `buf`
    auto arrive = [&](uint32_t buf) {
        if (buf ? bulk1 : bulk0) {
            if (!mbar_wait(&sh.bar[buf], (buf ? fills1 : fills0) & 1u)) status |= kStTimeout;
            if (buf) ++fills1; else ++fills0;
        }
        if (buf) bulk1 = false; else bulk0 = false;
        __syncwarp();
    };

    // the job of the tile looked up last: consecutive look-ups mostly stay inside it
    int cj = -1;
    uint32_t cj_begin = 0, cj_count = 0;
    const float* cj_x = nullptr;
    unsigned long long cj_n = 0;
    auto locate = [&](uint32_t t) {
        TileInfo ti;
        ti.job = -1; ti.tile = 0; ti.tiles = 1; ti.len = 0; ti.xt = nullptr; ti.mapped = false;
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
            ti.mapped = (((uintptr_t)cj_x) & 15u) == 0;
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

    uint32_t ticket = take_ticket(ws, lane);
    TileInfo cur = locate(ticket);
    uint32_t p = 0;   // stage that holds (or will hold) the round about to be encoded
    request(p, cur, 0);

    while (cur.job >= 0) {
        const uint32_t tile_begin = ticket - cur.tile;
        const uint32_t len = cur.len;
        const uint32_t nb = (len + kBlock - 1) / kBlock;
        const uint32_t padw = (nb + 3) >> 2;
        const uint32_t rounds = (nb + 31) >> 5;
        const uint32_t dir = pend.dir ^ 1u;   // the end of the blob area the waiting tile does not use
        const uint32_t org = dir ? (uint32_t)kEncBlobWords - 1u : 0u;
        const int sgn = dir ? -1 : 1;

        // the number of the tile after this one is asked for now and looked at in the last round
        uint32_t next_raw = 0;
        if (lane == 0) next_raw = atomicAdd(ws.ticket, 1u);
        uint32_t next = 0;
        TileInfo nxt;
        nxt.job = -1; nxt.tile = 0; nxt.tiles = 1; nxt.len = 0; nxt.xt = nullptr; nxt.mapped = false;

        EncodeCarry cy;
        cy.pay_used = 0; cy.wide = false;
        float carry_x = 0.0f;
        int32_t q_first = 0;
        bool general = false;
        // a tile without elements runs the loop once, for the hand-over to the next tile only
        for (uint32_t rd = 0; rd < (rounds ? rounds : 1u); ++rd) {
            __syncwarp();   // every lane is done with the other stage (it held the round before this one)
            const bool last_round = rd + 1 >= rounds;
            if (last_round) {
                next = __shfl_sync(kFull, next_raw, 0);
                nxt = locate(next);
                request(p ^ 1u, nxt, 0);
            } else {
                request(p ^ 1u, cur, (rd + 1) * kRound);
            }
            if (rounds == 0) break;
            // one window of the waiting tile's look-back rides along with this round
            const bool looking = pend.valid && !look_back_done(pend.lb);
            LookBackTrip<1> trip;
            if (looking) look_back_issue(ws, pend.lb, epoch, lane, trip);
            arrive(p);   // the round has landed
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
                                  lane, status, [] {});
                if (rc != 2 || !pend.valid) break;
                flush_pending();   // no room next to the waiting tile: place that one now, then try again
            }
            if (looking && pend.valid) (void)look_back_eval(ws, pend.lb, epoch, lane, trip);
            p ^= 1u;
            if (rc != 0) {
                general = true;
                if (!last_round) {   // hand over to the next tile: its first round goes where this tile's next round was asked into
                    arrive(p);   // this tile's next round, asked for above and not needed any more
                    next = __shfl_sync(kFull, next_raw, 0);
                    nxt = locate(next);
                    request(p, nxt, 0);
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
            LookBack lb_cur;
            look_back_begin(lb_cur, ticket, total, cur.job, tile_begin, cur.tiles);
            unsigned long long acc_old = ~0ull;
            if (lane == 0) {
                publish_tile_state(ws, ticket, total, epoch);
                acc_old = publish_size_issue(ws, lb_cur);
            }
            __syncwarp();   // the blob's words, written by all lanes, are visible to all
            if (lane == 0) publish_size_finish(ws, lb_cur, acc_old, epoch);   // before any wait: others may need the group's size
            if (pend.valid) flush_pending();
            pend.valid = true; pend.job = cur.job; pend.dir = dir;
            pend.lb = lb_cur;
            if (look_back_done(pend.lb)) look_back_publish(ws, pend.lb, epoch, lane);   // the job's first tile
        }
        cur = nxt;
        ticket = next;
    }
    if (pend.valid) flush_pending();
    if (status) atomicOr(ws.status, status);
    finish_launch(ws, epoch, tid, ws.ticket, (jb.total_tiles >> 5) + (uint32_t)jb.count + 1u);
}

// ------------------------------------------------------------------------------------------------ compress, two steps
//
// Step 1 (encode_rounds_kernel): the unit of work is a ROUND (32 blocks of a tile, one per lane).  A round needs
// nothing from the rounds around it but the element in front of it, so the rounds of a launch are handed to the warps
// by a counter in any order and nobody waits for anybody: a warp brings its round in with one tensor copy, encodes it
// into its shared memory and sends it off with one bulk store to the round's fixed slot in the workspace (code-length
// bytes, then payload), together with its size and, for a tile's first round, the tile's first quantised value.
// Step 2 (place_kernel) turns the slots into the stream.

constexpr int kRoundBufWords = 8 + 32 * 17;   // code-length bytes + payload at code length 16 (longer codes go the general route)
constexpr int kRoundStages = 3;
struct alignas(1024) RoundWarpShared {
    float stage[kRoundStages][kRound];        // each on a 1024-byte boundary; a round is encoded in place and leaves from here
    alignas(16) float front[kRoundStages][4]; // the four elements in front of each stage's round
    alignas(8) unsigned long long bar[kRoundStages];
};
static_assert(sizeof(RoundWarpShared) == 13 * 1024, "a warp's share of the shared memory");

// General route for one round: any code length, straight from global memory into the round's slot.
__device__ __noinline__ uint32_t encode_round_general(const float* __restrict__ xt, uint32_t len, uint32_t rd, float r, uint32_t* __restrict__ slot,
                                                      uint32_t* round_words, int32_t* outlier, unsigned long long* group_words, int lane)
{
    uint32_t status = 0;
    const uint32_t nb = (len + kBlock - 1) / kBlock;
    const uint32_t bi = 32u * rd + (uint32_t)lane;
    uint32_t planes[33];
    float tmax = 0.0f;
    uint32_t L = 0;
    if (bi < nb) L = general_block(xt, bi, len, r, planes, &tmax);
    if (!(tmax < 1073741824.0f)) status |= kStRange;
    else if (tmax > 32768.5f) status |= kStPrecision;
    const uint32_t nw = L ? L + 1u : 0u;
    const uint32_t incl = warp_incl_scan(nw, lane);
    reinterpret_cast<unsigned char*>(slot)[lane] = (unsigned char)L;
    if (L) {
        uint32_t* d = slot + 8 + (incl - nw);
        for (uint32_t k = 0; k <= L; ++k) d[k] = planes[k];
    }
    if (lane == 31) { *round_words = incl; atomicAdd(group_words, (unsigned long long)incl); }
    if (rd == 0 && lane == 0) *outlier = __float2int_rn(__fmul_rn(__ldg(xt), r));
    return status;
}

// The same for a round whose values sit in a stage (the hop's sums): block `lane` of the round from the lane's row.
__device__ __noinline__ uint32_t encode_round_general_staged(const float* stage, float xprev, bool active, uint32_t rd, float r,
                                                             uint32_t* __restrict__ slot, uint32_t* round_words, int32_t* outlier,
                                                             unsigned long long* group_words, int lane)
{
    uint32_t status = 0;
    const char* row = reinterpret_cast<const char*>(stage) + 128 * lane;
    const uint32_t sw = ((uint32_t)lane & 7u) << 4;
    uint32_t m[32];
    uint32_t sg = 0, ob = 0;
    const float tp = __fmul_rn(xprev, r);
    float tm = fabsf(tp);
    uint32_t qp = (uint32_t)__float2int_rn(tp);
    const int32_t q0 = __float2int_rn(__fmul_rn(*reinterpret_cast<const float*>(row + sw), r));
#pragma unroll
    for (int j = 0; j < 32; ++j) {
        const float x = *reinterpret_cast<const float*>(row + ((16u * (uint32_t)(j >> 2)) ^ sw) + 4 * (j & 3));
        const float tt = __fmul_rn(x, r);
        tm = fmaxf(tm, fabsf(tt));
        const uint32_t q = (uint32_t)__float2int_rn(tt);
        const int32_t dd = (int32_t)(q - qp);
        qp = q;
        const uint32_t sm = (uint32_t)(dd >> 31);
        m[j] = (((uint32_t)dd ^ sm) - sm) & 0x7FFFFFFFu;
        ob |= m[j];
        sg = __funnelshift_l((uint32_t)dd, sg, 1);
    }
    uint32_t L = active ? code_length(ob) : 0u;
    if (active) {
        if (!(tm < 1073741824.0f)) status |= kStRange;
        else if (tm > 32768.5f) status |= kStPrecision;
    }
    bit_transpose<32>(m);
    const uint32_t nw = L ? L + 1u : 0u;
    const uint32_t incl = warp_incl_scan(nw, lane);
    reinterpret_cast<unsigned char*>(slot)[lane] = (unsigned char)L;
    if (L) {
        uint32_t* d = slot + 8 + (incl - nw);
        d[0] = __brev(sg);
#pragma unroll
        for (int k = 0; k < 31; ++k)
            if ((uint32_t)k < L) d[1 + k] = m[k];
    }
    if (lane == 31) { *round_words = incl; atomicAdd(group_words, (unsigned long long)incl); }
    if (rd == 0 && lane == 0) *outlier = q0;
    return status;
}

// What a warp has to know of a tile when it gets to encode its round.
struct RoundAt {
    uint32_t t;          // launch number of the tile (beyond the launch: done)
    uint32_t len;        // elements of the tile (0: nothing to encode)
    uint32_t gslot;      // slot of the accumulator of the tile's group
    const float* xt;     // the tile's first element
};

// A warp's walk over the tiles of a launch, G tiles at a time: where the tile is and how long.
struct TileCursor {
    uint32_t t;          // launch number of the tile (beyond the launch: done)
    int job;
    uint32_t begin, count;   // the job's first tile and its number of tiles
    uint32_t len;        // elements of the tile (0: nothing to encode)
    const float* xt;     // the tile's first element
    bool aligned;        // the job's array starts on a 16-byte boundary
};

__device__ __forceinline__ void cursor_settle(TileCursor& c, const JobBatch& jb, bool valid)
{
    c.len = 0;
    if (c.t >= jb.total_tiles) return;
    if (c.t - c.begin >= c.count) {
        c.job = find_job(jb, c.t);
        c.begin = jb.job[c.job].tile_begin;
        c.count = (c.job + 1 < jb.count ? jb.job[c.job + 1].tile_begin : jb.total_tiles) - c.begin;
        c.aligned = (((uintptr_t)jb.job[c.job].x) & 15u) == 0;
    }
    const Job& q = jb.job[c.job];
    const unsigned long long start = (unsigned long long)(c.t - c.begin) * kTile;
    if (q.n && valid) {
        c.len = (uint32_t)((q.n - start < (unsigned long long)kTile) ? (q.n - start) : kTile);
        c.xt = q.x + start;
    }
}

__global__ void __launch_bounds__(kCodecThreads, 4) encode_rounds_kernel(const __grid_constant__ JobBatch jb, const __grid_constant__ TileMaps maps,
                                                                         Workspace ws, Params hp, int use_dev_params)
{
    // Before the kernel in front on the stream is waited for: the warp's first two rounds are asked into L2.  (A prefetch
    // only moves lines into L2, which stays coherent with whatever that kernel still writes.)
    if ((threadIdx.x & 31) == 0) {
        const uint32_t rd0 = threadIdx.x >> 5;
        for (uint32_t t = blockIdx.x, k = 0; k < 2 && t < jb.total_tiles; ++k, t += gridDim.x) {
            const int j = find_job(jb, t);
            const Job& q = jb.job[j];
            const unsigned long long e = (unsigned long long)(t - q.tile_begin) * kTile + (unsigned long long)rd0 * kRound;
            if (q.x && (((uintptr_t)q.x) & 15u) == 0 && e + kRound <= q.n) bulk_prefetch_l2(q.x + e, 4u * kRound);
        }
    }
    pdl_enter();
    extern __shared__ __align__(16) unsigned char smem_raw[];
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    RoundWarpShared& sh = reinterpret_cast<RoundWarpShared*>(smem_raw + ((1024u - (smem_u32(smem_raw) & 1023u)) & 1023u))[warp];
    uint32_t status = 0;
    Params prm = hp;
    if (use_dev_params) prm = *ws.params;
    const float r = prm.r;

    if (lane == 0) {
#pragma unroll
        for (int k = 0; k < kRoundStages; ++k) mbar_init(&sh.bar[k], 1);
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    __syncwarp();

    // The CTA's four warps take the four rounds of the same tile, and the CTAs of the launch take the tiles in turn
    // (no counter: same-address atomics would bound the kernel at about 1.5 ns per round).
    const uint32_t G = gridDim.x;
    const uint32_t rd = (uint32_t)warp, e0 = rd * (uint32_t)kRound;
    const uint32_t sw = ((uint32_t)lane & 7u) << 4;

    // Asks for the warp's round of the tile under cursor `c` into stage `st`.  Every request completes one phase of the
    // stage's mbarrier, whatever its kind: a tensor copy (with a 16-byte copy of the words in front, whose last one
    // is the element in front of the round), plain loads, or nothing at all.
    auto request = [&](const TileCursor& c, uint32_t st) {
        float* stage = sh.stage[st];
        if (c.t < jb.total_tiles && e0 < c.len) {
            if (c.aligned && e0 + (uint32_t)kRound <= c.len) {
                if (lane == 0) {
                    mbar_expect_tx(&sh.bar[st], kRound * 4 + (rd ? 16u : 0u));
                    asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
                    asm volatile("cp.async.bulk.tensor.2d.shared::cluster.global.tile.mbarrier::complete_tx::bytes [%0], [%1, {%2, %3}], [%4];"
                                 ::"r"(smem_u32(stage)), "l"(&maps.m[c.job]), "r"(0), "r"((int)((c.t - c.begin) * (uint32_t)kBlocksPerTile + (e0 >> 5))),
                                   "r"(smem_u32(&sh.bar[st])) : "memory");
                    if (rd)
                        asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], 16, [%2];"
                                     ::"r"(smem_u32(sh.front[st])), "l"(c.xt + e0 - 4), "r"(smem_u32(&sh.bar[st])) : "memory");
                }
                return;
            }
            load_round_ragged(stage, c.xt, e0, c.len, lane);
            if (lane == 0 && rd) sh.front[st][3] = __ldg(c.xt + e0 - 1u);
            __syncwarp();
        }
        if (lane == 0) mbar_arrive(&sh.bar[st]);
    };

    TileCursor ahead;   // the tile two steps on, whose round is asked for while the current one is encoded
    ahead.t = blockIdx.x; ahead.job = 0; ahead.begin = 0; ahead.count = 0; ahead.len = 0; ahead.xt = nullptr; ahead.aligned = false;
    auto at = [&](const TileCursor& c) {
        RoundAt a;
        a.t = c.t; a.len = c.len; a.xt = c.xt;
        a.gslot = (c.begin >> 5) + (uint32_t)c.job + ((c.t - c.begin) >> 5);
        return a;
    };
    auto step = [&]() {
        ahead.t = ahead.t + G < ahead.t ? 0xFFFFFFFFu : ahead.t + G;
        cursor_settle(ahead, jb, prm.valid != 0);
    };
    cursor_settle(ahead, jb, prm.valid != 0);
    RoundAt cur = at(ahead);
    request(ahead, 0);
    step();
    RoundAt nxt = at(ahead);
    request(ahead, 1);
    step();

    uint32_t st = 0, st2 = 2, phase = 0;   // stage of the current round, stage of the request, parity of the current stage's phase
    EncodeCarry cy;
    cy.pay_used = 0; cy.wide = false;

    while (cur.t < jb.total_tiles) {
        const uint32_t u = 4u * cur.t + rd;
        const uint32_t nb = (cur.len + kBlock - 1) / kBlock;
        if (!mbar_wait(&sh.bar[st], phase)) status |= kStTimeout;
        // the stage two steps on was encoded in place and sent off in the step before: the copy engine has to be through
        // with it before the next request lands there; by the time the rows are read and sized it mostly is
        auto mid = [&]() {
            if (lane == 0) asm volatile("cp.async.bulk.wait_group.read 0;" ::: "memory");
            __syncwarp();
            request(ahead, st2);
        };
        if (32u * rd < nb) {
            uint32_t* slot = ws.slots + (size_t)u * kRoundSlotWords;
            float* stage = sh.stage[st];
            const char* row = reinterpret_cast<const char*>(stage) + 128 * lane;
            const float first = stage[0];
            const float xprev = lane ? read_last_of_row(stage, (uint32_t)lane - 1u) : (rd ? sh.front[st][3] : first);
            const uint32_t gslot = cur.gslot;
            cy.pay_used = 0;
            // in place: the stage becomes the round's slot image (code-length bytes at words 0.., payload at word 8), laid
            // out like a tile's blob whose word 0 sits in front of it
            const int rc = encode_round(row, sw, xprev, r, 32u * rd + (uint32_t)lane < nb, (uint32_t)lane, 32u, reinterpret_cast<uint32_t*>(stage) - 1,
                                        0u, 1, 9u, (uint32_t)kRoundBufWords - 8u, cy, lane, status, mid);
            if (rc == 0) {
                __syncwarp();   // the words written by all lanes are visible to lane 0's store
                if (lane == 0) {
                    const uint32_t bytes = (32u + 4u * cy.pay_used + 15u) & ~15u;
                    asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
                    asm volatile("cp.async.bulk.global.shared::cta.bulk_group [%0], [%1], %2;" ::"l"(slot), "r"(smem_u32(stage)), "r"(bytes) : "memory");
                    asm volatile("cp.async.bulk.commit_group;" ::: "memory");
                    ws.round_words[u] = cy.pay_used;
                    atomicAdd(ws.group_acc + gslot, (unsigned long long)cy.pay_used);
                    // exact while |x r| < 2^22; larger codes take the general route
                    if (rd == 0) ws.outliers[cur.t] = (int32_t)(__float_as_uint(__fadd_rn(__fmul_rn(first, r), kRoundMagic)) - kRoundMagicBits);
                }
            } else {
                status |= encode_round_general(cur.xt, cur.len, rd, r, slot, ws.round_words + u, ws.outliers + cur.t, ws.group_acc + gslot, lane);
            }
        } else {
            mid();
            if (lane == 0) ws.round_words[u] = 0;   // a round beyond the tile's last block, or a tile without elements
        }
        cur = nxt;
        nxt = at(ahead);
        step();
        st2 = st;
        st = st == (uint32_t)kRoundStages - 1u ? 0u : st + 1u;
        if (st == 0) phase ^= 1u;
    }
    if (lane == 0) asm volatile("cp.async.bulk.wait_group 0;" ::: "memory");   // the stores have read shared memory and are complete
    if (status) atomicOr(ws.status, status);
}

// Step 2: one CTA per group of 32 tiles of a job turns the group's round slots into its piece of the stream.  The
// tiles' sizes follow from the rounds' sizes; the group's position is the sum of the groups of the job in front of
// it, found by a decoupled look-back over the group states (every CTA publishes its group's size as soon as it has
// read 128 numbers, so the waits are short; they are bounded all the same); then each warp copies tiles.
struct GroupTable {
    uint32_t begin[kMaxJobs + 1];   // first group (= CTA) of each job; begin[count] = number of groups
};
constexpr int kPlaceThreads = 1024;   // one warp per tile of the group
constexpr int kPlaceHeadWords = 288;  // payload words of a round that are fetched before its size is known (code lengths up to 8 on average); measured best of 192 ... 448
constexpr size_t kPlaceSmemBytes = (size_t)(kPlaceThreads / 32) * kRoundsPerTile * kPlaceHeadWords * 4;

// Called by one warp of every CTA of the placement once the CTA has read the group sums it needs: the last CTA to
// get there re-arms the workspace (group sums back to zero, launch counter on) while the others are still storing.
// `used`: group sums the launch may have touched.
__device__ __forceinline__ void rearm_groups(uint32_t used, const Workspace& ws, uint32_t epoch, int lane)
{
    uint32_t last = 0;
    if (lane == 0) {
        __threadfence();
        last = atomicAdd(ws.done, 1u) == gridDim.x - 1 ? 1u : 0u;
    }
    if (!__shfl_sync(kFull, last, 0)) return;
    for (uint32_t k = (uint32_t)lane; k < used; k += 32u) ws.group_acc[k] = 0ull;
    const uint32_t e = (epoch + 1u) & 0x7FFFFFFFu;
    if (e == 0) {   // the counter wraps (once in 2^31 launches): no scan state of an earlier launch may look current again
        for (uint32_t k = (uint32_t)lane; k < ws.max_tiles; k += 32u) st_state(ws.tile_state + k, 0ull);
        for (uint32_t k = (uint32_t)lane; k < (uint32_t)group_slots(ws.max_tiles); k += 32u) st_state(ws.group_state + k, 0ull);
        __threadfence();
    }
    __syncwarp();
    if (lane == 0) {
        *ws.done = 0;
        *ws.ticket = 0;
        *ws.epoch = e ? e : 1u;
    }
}

__device__ __forceinline__ void rearm_after_reads(const JobBatch& jb, const Workspace& ws, uint32_t epoch, int lane)
{
    rearm_groups((jb.total_tiles >> 5) + (uint32_t)jb.count + 1u, ws, epoch, lane);
}

// from_stream: 0 = a compression (bound in hp, or on the device), 1 = a hop (bound and step from the incoming stream's
// header), 2 = a compression of binary64 input (bound in hp64, or on the device; the header carries the step as one
// binary64).
__global__ void __launch_bounds__(kPlaceThreads) place_kernel(const __grid_constant__ JobBatch jb, const __grid_constant__ GroupTable gt, Workspace ws,
                                                              Params hp, int use_dev_params, int from_stream, ParamsF64 hp64)
{
    // What this kernel reads before it waits for step 1 is older than step 1's launch: job table, the incoming
    // streams' headers, the resolved bound.
    __shared__ uint32_t s_words[32], s_part[kPlaceThreads / 32];
    __shared__ alignas(8) unsigned long long s_bar[kPlaceThreads / 32];
    extern __shared__ __align__(16) unsigned char place_smem[];   // per warp: the first 1024 payload bytes of its tile's four rounds
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    uint32_t* stage = reinterpret_cast<uint32_t*>(place_smem) + (size_t)warp * (kRoundsPerTile * kPlaceHeadWords);
    if (lane == 0) {
        mbar_init(&s_bar[warp], 1);
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    __syncwarp();
    uint32_t status = 0;
    Params prm = hp;
    double step64 = hp64.s;
    if (from_stream == 2) {
        if (use_dev_params) { const ParamsF64 p = *ws.params64; step64 = p.s; prm.valid = p.valid; }
        else prm.valid = hp64.valid;
    } else if (use_dev_params) prm = *ws.params;
    auto put_header = [&](uint32_t* out, int who, unsigned long long n, uint32_t nT) {
        if (from_stream != 2) { write_header(out, who, n, prm.eb_abs, prm.s, nT); return; }
        if (who < kHeaderWords) {
            const uint32_t words[kHeaderWords] = {kMagic, kVersionF64, (uint32_t)n, (uint32_t)(n >> 32), (uint32_t)__double2loint(step64),
                                                  (uint32_t)__double2hiint(step64), (uint32_t)kTile, nT};
            uint32_t hv = words[0];
#pragma unroll
            for (int k = 1; k < kHeaderWords; ++k) hv = who == k ? words[k] : hv;
            out[who] = hv;
        }
    };

    int j = 0;
    {
        int lo = 0, hi = jb.count;
        while (hi - lo > 1) {
            const int mid = (lo + hi) >> 1;
            if (gt.begin[mid] <= blockIdx.x) lo = mid; else hi = mid;
        }
        j = lo;
    }
    const Job& job = jb.job[j];
    if (from_stream == 1) {   // a hop: bound and step are the incoming stream's, and the job counts only if its streams agree with it
        const StreamInfo h1 = read_header(job.in_c, job.in_cap);
        bool ok = h1.ok && h1.n == job.n;
        if (job.in_c2) {
            const StreamInfo h2 = read_header(job.in_c2, job.in2_cap);
            ok = ok && h2.ok && h2.n == job.n && __float_as_uint(h2.s) == __float_as_uint(h1.s);
        }
        prm.eb_abs = h1.eb_abs; prm.s = h1.s; prm.valid = ok ? 1 : 0;
    }
    pdl_enter();
    const uint32_t epoch = *reinterpret_cast<volatile uint32_t*>(ws.epoch);
    const uint32_t g = blockIdx.x - gt.begin[j];
    const uint32_t tiles = (j + 1 < jb.count ? jb.job[j + 1].tile_begin : jb.total_tiles) - job.tile_begin;
    const unsigned long long n = job.n;
    const uint32_t nT = (uint32_t)((n + kTile - 1) / kTile);
    uint32_t* __restrict__ out = job.out;

    if (n == 0 || !prm.valid) {   // a job without elements, or no valid bound: header and length only
        const bool hdr = prm.valid && job.out_cap >= (unsigned)kHeaderBytes;
        if (tid == 0) *job.out_bytes = hdr ? kHeaderBytes : 0;
        if (hdr) put_header(out, tid, 0, 0);
        if (warp == kPlaceThreads / 32 - 1) rearm_after_reads(jb, ws, epoch, lane);
    } else {
        const uint32_t t0 = 32u * g;                               // first tile of the group, within the job
        const uint32_t ntl = tiles - t0 < 32u ? tiles - t0 : 32u;   // tiles of the group
        const uint32_t T0 = job.tile_begin + t0;                   // the same, in the launch's numbering
        // One round trip: every warp asks for all that belongs to its tile at once (round sizes, first value, its lane's
        // code-length word, eight payload words per lane and round whatever the sizes turn out to be) and for its share of
        // the sums of the groups in front.
        const uint32_t tl = (uint32_t)warp;
        const bool mine = tl < ntl;
        const uint32_t T = T0 + (mine ? tl : 0u);
        const uint32_t* __restrict__ slot = ws.slots + (size_t)(4u * T) * kRoundSlotWords;
        const uint4 nq4 = *reinterpret_cast<const uint4*>(ws.round_words + 4u * T);
        const uint32_t lword = slot[(size_t)(lane >> 3) * kRoundSlotWords + (lane & 7)];   // code-length word `lane` of the tile
        const uint32_t first = (uint32_t)ws.outliers[T];
        if (mine && lane == 0) {   // the copy engine brings the heads of the four payloads: four requests instead of 32 loads per lane
            mbar_expect_tx(&s_bar[warp], kRoundsPerTile * kPlaceHeadWords * 4);
#pragma unroll
            for (int q = 0; q < kRoundsPerTile; ++q)
                bulk_load(stage + q * kPlaceHeadWords, slot + (size_t)q * kRoundSlotWords + 8, kPlaceHeadWords * 4, &s_bar[warp]);
        }
        unsigned long long part = 0;
        {
            const uint32_t gslot0 = (job.tile_begin >> 5) + (uint32_t)j;
            for (uint32_t k = (uint32_t)tid; k < g; k += kPlaceThreads) part += ws.group_acc[gslot0 + k];
        }
        const uint32_t nqs[kRoundsPerTile] = {nq4.x, nq4.y, nq4.z, nq4.w};
        {
            const unsigned long long left = n - (unsigned long long)(t0 + (mine ? tl : 0u)) * kTile;
            const uint32_t len = (uint32_t)(left < (unsigned long long)kTile ? left : (unsigned long long)kTile);
            const uint32_t padw = (((len + kBlock - 1) / kBlock) + 3) >> 2;
#pragma unroll
            for (int d = 16; d >= 1; d >>= 1) part += __shfl_xor_sync(kFull, part, d);
            if (lane == 0) {
                s_words[warp] = mine ? 1u + padw + nq4.x + nq4.y + nq4.z + nq4.w : 0u;
                s_part[warp] = (uint32_t)part;
            }
        }
        __syncthreads();
        if (warp == kPlaceThreads / 32 - 1) rearm_after_reads(jb, ws, epoch, lane);   // every warp's reads of the sums are through
        // the group's place: the groups of the job in front of it are full ones (33 fixed words per tile) with the
        // payload that step 1 added up per group; the tile's place inside the group: the tiles in front of it
        const uint32_t wl = s_words[lane];
        const uint32_t incl = warp_incl_scan(wl, lane);
        const uint32_t my_off = __shfl_sync(kFull, incl - wl, warp);
        const uint32_t base = __reduce_add_sync(kFull, s_part[lane]) + g * 32u * (1u + (uint32_t)kLWords);
        const bool placed = true;
        if (mine) {
            const uint32_t tile = t0 + tl;
            const uint32_t words = s_words[tl];
            const unsigned long long word0 = (unsigned long long)kHeaderWords + nT + base + my_off;
            const bool fits = (word0 + words) * 4ull <= job.out_cap;
            if (!fits) status |= kStCapacity;
            // the copies into this warp's shared memory land before anything else happens (also when the tile does not fit:
            // a CTA must not end with copies into its shared memory still on their way)
            if (!mbar_wait(&s_bar[warp], 0u)) status |= kStTimeout;
            if (fits && placed) {
                uint32_t* __restrict__ dst = out + word0;
                const unsigned long long tleft = n - (unsigned long long)tile * kTile;
                const uint32_t tlen = (uint32_t)(tleft < (unsigned long long)kTile ? tleft : (unsigned long long)kTile);
                const uint32_t tpadw = (((tlen + kBlock - 1) / kBlock) + 3) >> 2;
                if (lane == 0) dst[0] = first;
                if ((uint32_t)lane < tpadw) dst[1 + lane] = lword;
                uint32_t* __restrict__ d = dst + 1 + tpadw;
#pragma unroll
                for (int q = 0; q < kRoundsPerTile; ++q) {
                    const uint32_t nq = nqs[q];
#pragma unroll
                    for (int k = 0; k < kPlaceHeadWords / 32; ++k) {
                        const uint32_t i = (uint32_t)lane + 32u * k;
                        if (i < nq) d[i] = stage[q * kPlaceHeadWords + i];
                    }
                    if (nq > (uint32_t)kPlaceHeadWords) {   // code lengths beyond 7 on average: the rest of the round
                        const uint32_t* __restrict__ src = slot + (size_t)q * kRoundSlotWords + 8;
                        for (uint32_t i = (uint32_t)kPlaceHeadWords + (uint32_t)lane; i < nq; i += 32) d[i] = src[i];
                    }
                    d += nq;
                }
                if (lane == 0) out[kHeaderWords + tile] = base + my_off + words;
            }
            if (lane == 0 && tile == nT - 1) *job.out_bytes = (size_t)((word0 + words) * 4ull);
            if (tile == 0) put_header(out, lane, n, nT);
        }
    }
    if (status) atomicOr(ws.status, status);
}

// ------------------------------------------------------------------------------------------------ decompress
//
// A warp decodes a tile of its own in four rounds, lane l of a round taking block 32 * round + l: the block's sign
// word and planes come out of the tile's blob (staged in shared memory by a bulk copy, one tile ahead), the block's
// sum of deltas follows from population counts of the planes, a shuffle scan of those sums gives every block the
// code in front of it, and the lane then walks its 32 elements: inverse bit-matrix transpose, magnitude, sign,
// running code, one multiplication; the values go into the lane's row of a swizzled stage, which one tiled tensor
// store (or, for ragged ends and unaligned arrays, a loop of coalesced stores) moves to the output.

// What a tile's code-length bytes say, found by every lane alike: 0 = inconsistent with the blob's size (or a code
// length above 31, or a non-zero padding byte), 1 = consistent and every code of the tile stays below 2^23 in
// magnitude (fp32 arithmetic is exact), 2 = consistent, integer arithmetic needed.  blob: the tile's words.
__device__ __forceinline__ int describe_blob(const uint32_t* blob, uint32_t words, uint32_t nb, int lane)
{
    const uint32_t padw = (nb + 3) >> 2;
    if (words < 1u + padw) return 0;
    const uint32_t lw = (uint32_t)lane < padw ? blob[1 + lane] : 0u;
    const uint32_t L0 = lw & 0xFFu, L1 = (lw >> 8) & 0xFFu, L2 = (lw >> 16) & 0xFFu, L3 = lw >> 24;
    bool bad = (lw & 0xE0E0E0E0u) != 0u;   // a code length above 31
    const uint32_t b0 = 4u * (uint32_t)lane;   // blocks at or beyond nb are padding of the code-length area: must be zero
    if ((b0 + 0 >= nb && L0) || (b0 + 1 >= nb && L1) || (b0 + 2 >= nb && L2) || (b0 + 3 >= nb && L3)) bad = true;
    const uint32_t sizes = (L0 ? L0 + 1 : 0) + (L1 ? L1 + 1 : 0) + (L2 ? L2 + 1 : 0) + (L3 ? L3 + 1 : 0);
    const uint32_t total = __reduce_add_sync(kFull, sizes);
    // every partial sum of deltas is below sum_b 32 * 2^L_b; with the outlier it must stay below 2^24
    const uint32_t Lmax = max(max(L0, L1), max(L2, L3));
    uint32_t spread = 1u << 24;
    if (Lmax <= 18u) spread = (32u << L0) + (32u << L1) + (32u << L2) + (32u << L3);
    spread = __reduce_add_sync(kFull, min(spread, 1u << 24));   // at most 32 * 2^24 = 2^29: no overflow
    if (__any_sync(kFull, bad) || 1u + padw + total != words) return 0;
    const int32_t outlier = (int32_t)blob[0];
    const uint32_t ao = (uint32_t)(outlier < 0 ? -outlier : outlier);
    return (ao < (1u << 23) && spread < (1u << 23)) ? 1 : 2;
}

// A block's sign word and planes (payload words pay[0 .. L]) as N-bit packed words ready for the inverse transpose,
// N = 8, 16 or 32 (code lengths up to N), and the block's sum of deltas.
template <int N>
__device__ __forceinline__ int32_t load_planes(const uint32_t* pay, uint32_t L, uint32_t& sign, uint32_t (&w)[N])
{
    sign = L ? pay[0] : 0u;
    int32_t total = 0;
#pragma unroll
    for (int k = 0; k < N; ++k) {
        w[k] = (uint32_t)k < L ? pay[1 + k] : 0u;
        // elements with the bit set count 2^k each, negative ones with the opposite sign
        total += (__popc(w[k]) - 2 * __popc(w[k] & sign)) << k;
    }
    return total;
}

// The lane's 32 elements from the transposed words (word i, field h = magnitude of element N h + i), written as
// values into the lane's row of a stage.  Codes are exact in fp32 (the caller checked): the magnitude is read as a
// float from its bits, gets its sign, joins the running code, and one multiplication makes the value.  MODE 0:
// plain decoding; MODE 1: every value is added to the operand in the same place of the row `loc`.
template <int N, int MODE>
__device__ __forceinline__ void expand_block(const uint32_t (&w)[N], uint32_t sign, int32_t code_in_front, float s, char* row, uint32_t sw,
                                             const char* loc)
{
    float run = (float)code_in_front;
    uint32_t sel = N == 8 ? 0x7650u : 0x7610u;   // byte (pair) h of a word under the exponent of 2^23
#pragma unroll 1
    for (int h = 0; h < 32 / N; ++h) {
#pragma unroll
        for (int q = 0; q < N / 4; ++q) {
            float o[4];
            const uint32_t at = (16u * (uint32_t)(h * (N / 4) + q)) ^ sw;
            if (MODE == 1) {
                // the hop: the magnitudes and the products go two elements to an instruction (sm_100's packed fp32, each half
                // rounded as the scalar operation is); the running code stays a chain of scalar additions, and the sums with the
                // operand stay scalar too: the compiler contracts a packed product and a packed addition behind it into a
                // packed fused multiply-add whatever --fmad says, and Eq. 2 adds to the ROUNDED decompressed value.
                // 43.1 -> 42.4 us per 64 MiB.  The plain decoder gains nothing from packing and keeps the scalar form.
                const float2 neg23 = make_float2(-kTwo23, -kTwo23), s2 = make_float2(s, s);
                const float2 m01 = __fadd2_rn(make_float2(__uint_as_float(prmt(w[4 * q + 0], 0x4B000000u, sel)),
                                                          __uint_as_float(prmt(w[4 * q + 1], 0x4B000000u, sel))), neg23);
                const float2 m23 = __fadd2_rn(make_float2(__uint_as_float(prmt(w[4 * q + 2], 0x4B000000u, sel)),
                                                          __uint_as_float(prmt(w[4 * q + 3], 0x4B000000u, sel))), neg23);
                const float ms[4] = {m01.x, m01.y, m23.x, m23.y};
                float rs[4];
#pragma unroll
                for (int e = 0; e < 4; ++e) {
                    const int i = 4 * q + e;
                    const uint32_t sbit = (sign << (31 - i)) & 0x80000000u;
                    run = __fadd_rn(run, __uint_as_float(__float_as_uint(ms[e]) | sbit));
                    rs[e] = run;
                }
                const float4 l = *reinterpret_cast<const float4*>(loc + at);
                const float2 p01 = __fmul2_rn(make_float2(rs[0], rs[1]), s2), p23 = __fmul2_rn(make_float2(rs[2], rs[3]), s2);
                o[0] = __fadd_rn(p01.x, l.x); o[1] = __fadd_rn(p01.y, l.y); o[2] = __fadd_rn(p23.x, l.z); o[3] = __fadd_rn(p23.y, l.w);
            } else {
#pragma unroll
                for (int e = 0; e < 4; ++e) {
                    const int i = 4 * q + e;
                    const float m = __fsub_rn(__uint_as_float(prmt(w[i], 0x4B000000u, sel)), kTwo23);
                    const uint32_t sbit = (sign << (31 - i)) & 0x80000000u;
                    run = __fadd_rn(run, __uint_as_float(__float_as_uint(m) | sbit));
                    o[e] = __fmul_rn(run, s);
                }
            }
            *reinterpret_cast<float4*>(row + at) = make_float4(o[0], o[1], o[2], o[3]);
        }
        sign >>= N;
        sel += N == 8 ? 0x0001u : 0x0022u;
    }
}

// Reduce operation of the hop: 0 = sum, 1 = max, 2 = min, 3 = average (a sum on every hop); of two operands that
// compare equal Max and Min keep the decoded one.
__device__ __forceinline__ float combine(uint32_t op, float a, float b)
{
    return op == 1u ? ((a < b) ? b : a) : op == 2u ? ((b < a) ? b : a) : __fadd_rn(a, b);
}

// Where a tile's blob is, as known from the index alone.
struct BlobRef {
    const uint32_t* ptr;    // nullptr: no blob (tile beyond the stream, or a stream that does not parse)
    uint32_t words;
    bool staged;            // a bulk copy of its 16-byte-aligned cover is on its way
};

// One round of a tile (blocks 32 rd + lane) by the general route: any code length, integer arithmetic, any reduce
// operation.  blob: the tile's words (shared or global memory); pay_off: payload words of the rounds before; code:
// the code in front of the round; loc_stage: the stage with the operand's round, or nullptr.  Leaves the values in
// `stage`.  Compact rather than fast: the rounds that come here are rare.
__device__ __noinline__ void decode_round_general(const uint32_t* blob, uint32_t padw, uint32_t L, uint32_t* pay_off_io, int32_t* code_io,
                                                  float s, float* stage, int lane, const float* loc_stage, uint32_t op)
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
    char* row = reinterpret_cast<char*>(stage) + 128 * lane;
    const char* loc = reinterpret_cast<const char*>(loc_stage) + 128 * lane;
    const uint32_t sw = ((uint32_t)lane & 7u) << 4;
#pragma unroll
    for (int j = 0; j < 32; ++j) {
        run += ((sign >> j) & 1u) ? -(int32_t)w[j] : (int32_t)w[j];
        float v = __fmul_rn(__int2float_rn(run), s);
        const uint32_t at = ((16u * (uint32_t)(j >> 2)) ^ sw) + 4u * (j & 3);
        if (loc_stage) v = combine(op, v, *reinterpret_cast<const float*>(loc + at));
        *reinterpret_cast<float*>(row + at) = v;
    }
}

constexpr int kDecBlobWords = 1024 + 8;   // blob buffers: a window of 4 KiB plus the slack of the 16-byte-aligned cover

// The code lengths of a lane's four blocks of a tile (blocks lane, 32 + lane, 64 + lane, 96 + lane), one per byte, from
// the head of the tile's blob: kept in a register, because the window over a large blob moves away from its head.
__device__ __forceinline__ uint32_t lane_code_lengths(const uint32_t* blob, uint32_t nb, int lane)
{
    const unsigned char* lb = reinterpret_cast<const unsigned char*>(blob + 1);
    uint32_t lp = 0;
#pragma unroll
    for (uint32_t e = 0; e < (uint32_t)kRoundsPerTile; ++e) {
        const uint32_t bi = 32u * e + (uint32_t)lane;
        if (bi < nb) lp |= (uint32_t)lb[bi] << (8u * e);
    }
    return lp;
}

// The window a warp has over its current tile's blob: words [0, end) of the blob can be read at base[word].  A blob
// that a bulk copy can bring (BlobRef::staged) is staged a window at a time: first its front, and when a round reaches
// past the window's end, the window moves to that round's first word.  Other blobs are read where they are.
struct BlobWindow {
    const uint32_t* base;
    uint32_t end;
};
// How much of a blob the copy that brings words [first, ...) covers: bytes to copy from the 16-byte boundary at or
// below that word (at most a buffer's worth, at most to the 16-byte boundary at or above the blob's end).
__device__ __forceinline__ uint32_t window_bytes(const BlobRef& br, uint32_t first)
{
    const uintptr_t g = (uintptr_t)(br.ptr + first), e = (uintptr_t)(br.ptr + br.words);
    const uintptr_t a_beg = g & ~(uintptr_t)15, a_end = (e + 15) & ~(uintptr_t)15;
    const uintptr_t bytes = a_end - a_beg;
    return (uint32_t)(bytes < (uintptr_t)(kDecBlobWords * 4) ? bytes : (uintptr_t)(kDecBlobWords * 4));
}
// The window after that copy has landed in `buf`.
__device__ __forceinline__ BlobWindow window_at(const BlobRef& br, uint32_t first, const uint32_t* buf)
{
    const uint32_t lead = (uint32_t)(((uintptr_t)(br.ptr + first)) & 15u) >> 2;   // words between the boundary and the first word
    BlobWindow w;
    w.base = buf + lead - first;
    const uint32_t got = first + (window_bytes(br, first) >> 2) - lead;
    w.end = got < br.words ? got : br.words;
    return w;
}
// Issues the copy (one lane).
__device__ __forceinline__ void window_request(const BlobRef& br, uint32_t first, uint32_t* buf, unsigned long long* bar)
{
    const uint32_t bytes = window_bytes(br, first);
    mbar_expect_tx(bar, bytes);
    bulk_load(buf, (const void*)(((uintptr_t)(br.ptr + first)) & ~(uintptr_t)15), bytes, bar);
}

// Tiled tensor store of a stage to rows [row0, row0 + 32) of the array behind `map` (one thread).
__device__ __forceinline__ void tensor_store_round(const CUtensorMap* map, uint32_t row0, const float* stage)
{
    asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
    asm volatile("cp.async.bulk.tensor.2d.global.shared::cta.tile.bulk_group [%0, {%1, %2}], [%3];"
                 ::"l"(map), "r"(0), "r"((int)row0), "r"(smem_u32(stage)) : "memory");
    asm volatile("cp.async.bulk.commit_group;" ::: "memory");
}
// The same for ragged ends and unaligned arrays: `count` elements of the stage, coalesced.
__device__ __noinline__ void store_round_ragged(float* __restrict__ y, const float* stage, uint32_t count, int lane)
{
#pragma unroll 4
    for (int k = 0; k < 32; ++k) {
        const uint32_t e = 32u * k + (uint32_t)lane;
        if (e < count) y[e] = *reinterpret_cast<const float*>(reinterpret_cast<const char*>(stage) + stage_chunk_byte(k, (uint32_t)lane >> 2) + 4 * (lane & 3));
    }
}

// One round of a tile whose codes are exact in fp32: blocks 32 rd + lane.  Arguments as for decode_round_general;
// MODE as for expand_block.  The lanes of a warp mostly share one width class; a round with a code length above 16
// takes the general route.
template <int N, int MODE>
__device__ __forceinline__ void decode_round_n(const uint32_t* blob, uint32_t padw, uint32_t L, uint32_t& pay_off, int32_t& code, float s,
                                               float* stage, int lane, const float* loc_stage)
{
    const uint32_t nw = L ? L + 1u : 0u;
    const uint32_t incl = warp_incl_scan(nw, lane);
    const uint32_t* pay = blob + 1 + padw + pay_off + (incl - nw);
    pay_off += __shfl_sync(kFull, incl, 31);
    char* row = reinterpret_cast<char*>(stage) + 128 * lane;
    const char* loc = reinterpret_cast<const char*>(loc_stage) + 128 * lane;
    const uint32_t sw = ((uint32_t)lane & 7u) << 4;
    // The block's sum of deltas first, so that the scan over the lanes gives the code in front of every block before
    // any element is expanded.
    uint32_t sign;
    uint32_t w[N];
    const int32_t total = load_planes<N>(pay, L, sign, w);
    int32_t inc = total;
#pragma unroll
    for (int d = 1; d < 32; d <<= 1) {
        const int32_t v = __shfl_up_sync(kFull, inc, d);
        if (lane >= d) inc += v;
    }
    bit_transpose<N>(w);
    expand_block<N, MODE>(w, sign, code + inc - total, s, row, sw, loc);
    code += __shfl_sync(kFull, inc, 31);
}
// The width class of round rd of a tile, the same for all lanes: 8, 16, or 0 when a code length above 16 sends the
// round down the general route.
__device__ __forceinline__ int round_class(uint32_t L)
{
    if (__any_sync(kFull, L > 16u)) return 0;
    return __any_sync(kFull, L > 8u) ? 16 : 8;
}
// The decoder's own form: one function with both classes (measured faster there than the two instantiations above
// behind a dispatch, which the hop uses out of line to keep its register count down).
// `ready` is called once by all lanes, after the planes are read and transposed and before the first value is stored:
// the place to make sure the stage is free.
template <int MODE, class Ready>
__device__ __forceinline__ void decode_round(const uint32_t* blob, uint32_t padw, uint32_t L, uint32_t& pay_off, int32_t& code, float s,
                                             float* stage, int lane, const float* loc_stage, Ready&& ready)
{
    if (__any_sync(kFull, L > 16u)) {
        ready();
        decode_round_general(blob, padw, L, &pay_off, &code, s, stage, lane, loc_stage, 0u);
        return;
    }
    const uint32_t nw = L ? L + 1u : 0u;
    const uint32_t incl = warp_incl_scan(nw, lane);
    const uint32_t* pay = blob + 1 + padw + pay_off + (incl - nw);
    pay_off += __shfl_sync(kFull, incl, 31);
    char* row = reinterpret_cast<char*>(stage) + 128 * lane;
    const char* loc = reinterpret_cast<const char*>(loc_stage) + 128 * lane;
    const uint32_t sw = ((uint32_t)lane & 7u) << 4;
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
        expand_block<8, MODE>(w, sign, code + inc - total, s, row, sw, loc);
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
        expand_block<16, MODE>(w, sign, code + inc - total, s, row, sw, loc);
        code += __shfl_sync(kFull, inc, 31);
    }
}
template <int MODE>
__device__ __forceinline__ void decode_round(const uint32_t* blob, uint32_t padw, uint32_t L, uint32_t& pay_off, int32_t& code, float s,
                                             float* stage, int lane, const float* loc_stage = nullptr)
{
    decode_round<MODE>(blob, padw, L, pay_off, code, s, stage, lane, loc_stage, [] {});
}

struct alignas(1024) DecWarpShared {
    float out[kRound];                     // one output stage
    alignas(16) uint32_t blob[2][kDecBlobWords];   // this tile's blob (or a window over it) and the next tile's
    alignas(8) unsigned long long bar[2];
};
static_assert(sizeof(DecWarpShared) == 13 * 1024, "a warp's share of the shared memory");
template <int CAP>
__global__ void __launch_bounds__(kCodecThreads, 4) decode_tiles_kernel(const __grid_constant__ JobBatchT<CAP> jb,
                                                                        const __grid_constant__ TileMapsT<CAP> maps, Workspace ws)
{
    pdl_enter();
    extern __shared__ __align__(16) unsigned char smem_raw[];
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    DecWarpShared& sh = reinterpret_cast<DecWarpShared*>(smem_raw + ((1024u - (smem_u32(smem_raw) & 1023u)) & 1023u))[warp];
    uint32_t status = 0;
    if (lane == 0) {
        mbar_init(&sh.bar[0], 1); mbar_init(&sh.bar[1], 1);
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    __syncwarp();
    uint32_t fills0 = 0, fills1 = 0;   // bulk copies completed into each blob buffer (phase parities of their mbarriers)
    uint32_t cb = 0;                   // the buffer with the current tile's blob

    // the job of the tile looked up last, with its stream's header
    int cj = -1;
    uint32_t cj_begin = 0, cj_count = 0;
    StreamInfo h;
    h.ok = false; h.n = 0; h.nT = 0; h.s = 1.0f; h.eb_abs = 0.0f;
    auto enter_job = [&](uint32_t t) {
        if (t - cj_begin >= cj_count) {
            cj = find_job(jb, t);
            const Job& q = jb.job[cj];
            cj_begin = q.tile_begin;
            cj_count = (cj + 1 < jb.count ? jb.job[cj + 1].tile_begin : jb.total_tiles) - cj_begin;
            h = read_header(q.in_c, q.in_cap);
        }
    };
    // The blob of tile t of the launch, from the index alone; the front of its 16-byte-aligned cover is requested into the
    // blob buffer when the cover lies inside the readable bytes.  Uniform over the warp.
    auto request = [&](uint32_t t, uint32_t buf) {
        BlobRef br;
        br.ptr = nullptr; br.words = 0; br.staged = false;
        if (t >= jb.total_tiles) return br;
        // the tile's index entries are asked for before the job's header is looked at (they need only the job table), so that
        // a warp's first tile waits for one round trip, not two
        uint32_t w_end = 0, w_beg = 0;
        {
            const bool same = t - cj_begin < cj_count;
            const int jn = same ? cj : find_job(jb, t);
            const Job& qn = jb.job[jn];
            const uint32_t tl = t - qn.tile_begin;
            if ((unsigned long long)kHeaderBytes + 4ull * ((unsigned long long)tl + 1ull) <= qn.in_cap) {
                const uint32_t* idx = qn.in_c + kHeaderWords;
                w_end = ldg_u32(idx + tl);
                w_beg = tl ? ldg_u32(idx + tl - 1) : 0u;
            }
        }
        enter_job(t);
        const Job& q = jb.job[cj];
        const uint32_t tile = t - cj_begin;
        if (!h.ok || h.n > q.n || tile >= h.nT) return br;
        const unsigned long long blob0 = (unsigned long long)kHeaderWords + h.nT;
        if (w_end <= w_beg || (blob0 + w_end) * 4ull > q.in_cap) { br.words = 0xFFFFFFFFu; return br; }   // marks a damaged index
        br.ptr = q.in_c + blob0 + w_beg;
        br.words = w_end - w_beg;
        const uintptr_t a_end = ((uintptr_t)(br.ptr + br.words) + 15) & ~(uintptr_t)15;
        if (a_end - (uintptr_t)q.in_c <= (uintptr_t)q.in_cap) {   // the copies may read up to the boundary behind the blob
            if (lane == 0) window_request(br, 0, sh.blob[buf], &sh.bar[buf]);
            br.staged = true;
        }
        return br;
    };

    const uint32_t stride = gridDim.x * (uint32_t)kCodecWarps;
    uint32_t t = blockIdx.x * (uint32_t)kCodecWarps + (uint32_t)warp;
    uint32_t so = 0;   // output stage to use next
    BlobRef cur = request(t, 0);
    while (t < jb.total_tiles) {
        // the current tile's facts, before the look-up of the next tile moves on to another job
        enter_job(t);
        const Job& job = jb.job[cj];
        const uint32_t tile = t - cj_begin;
        const StreamInfo hc = h;
        const int jcur = cj;
        const bool job_bad = !hc.ok, too_small = hc.ok && hc.n > job.n;
        const uint32_t tn = t + stride < t ? 0xFFFFFFFFu : t + stride;
        // Two blob buffers and ONE output stage in the 13 KiB that keep 16 warps on an SM: the next tile's blob is asked for
        // when this tile's has arrived, a whole tile ahead (with one buffer it was asked for after this tile's last round
        // and every tile began with a wait for it: 19.0 us per 64 MiB against 18.0), and the wait for the tensor store that
        // drains the stage sits behind the reading and transposing of the next round's planes, where it costs nothing.
        BlobRef nxt;
        nxt.ptr = nullptr; nxt.words = 0; nxt.staged = false;
        auto ask_next = [&]() {
            __syncwarp();   // every lane is done with the other blob buffer (the tile before)
            nxt = request(tn, cb ^ 1u);
        };
        if (cur.staged) {
            if (!mbar_wait(&sh.bar[cb], (cb ? fills1 : fills0) & 1u)) status |= kStTimeout;
            if (cb) ++fills1; else ++fills0;
        }
        ask_next();   // the other blob buffer takes the next tile's blob while this tile is decoded
        if (job_bad) status |= kStBadStream;
        else if (too_small) status |= kStCapacity;
        else if (cur.words == 0xFFFFFFFFu) status |= kStBadStream;
        else if (cur.ptr) {
            const unsigned long long start = (unsigned long long)tile * kTile;
            const uint32_t len = (uint32_t)((hc.n - start < (unsigned long long)kTile) ? (hc.n - start) : kTile);
            const uint32_t nb = (len + kBlock - 1) / kBlock, padw = (nb + 3) >> 2;
            BlobWindow win;
            win.base = cur.ptr; win.end = cur.words;
            if (cur.staged) win = window_at(cur, 0, sh.blob[cb]);
            const int mode = describe_blob(win.base, cur.words, nb, lane);   // the head (at most 33 words) is in every first window
            if (mode == 0) status |= kStBadStream;
            else {
                float* __restrict__ y = job.y + start;
                const bool mapped = (((uintptr_t)job.y) & 15u) == 0;
                uint32_t pay_off = 0;
                int32_t code = (int32_t)win.base[0];
                const uint32_t lp = lane_code_lengths(win.base, nb, lane);
                const uint32_t rounds = (nb + 31) >> 5;
                for (uint32_t rd = 0; rd < rounds; ++rd) {
                    const uint32_t L = (lp >> (8u * rd)) & 0xFFu;
                    const uint32_t first = 1u + padw + pay_off;
                    // only a blob larger than its buffer has a window that ends before the blob does
                    if (win.end < cur.words && first + __reduce_add_sync(kFull, L ? L + 1u : 0u) > win.end) {   // the round reaches past the window
                        __syncwarp();         // every lane is done with the window as it is
                        if (lane == 0) window_request(cur, first, sh.blob[cb], &sh.bar[cb]);
                        if (!mbar_wait(&sh.bar[cb], (cb ? fills1 : fills0) & 1u)) status |= kStTimeout;
                        if (cb) ++fills1; else ++fills0;
                        win = window_at(cur, first, sh.blob[cb]);
                    }
                    const uint32_t* blob = win.base;
                    // the stage about to be written was handed to a tensor store two rounds ago
                    // the one output stage was handed to a tensor store a round ago: by the time this round's planes are read and
                    // transposed the store has drained it
                    auto ready = [&]() {
                        if (lane == 0) asm volatile("cp.async.bulk.wait_group.read 0;" ::: "memory");
                        __syncwarp();
                    };
                    float* stage = sh.out;
                    if (mode == 1) decode_round<0>(blob, padw, L, pay_off, code, hc.s, stage, lane, nullptr, ready);
                    else { ready(); decode_round_general(blob, padw, L, &pay_off, &code, hc.s, stage, lane, nullptr, 0u); }
                    __syncwarp();   // the stage's rows, written by all lanes, are visible
                    const uint32_t e0 = rd * (uint32_t)kRound;
                    if (mapped && e0 + (uint32_t)kRound <= len) {
                        if (lane == 0) tensor_store_round(&maps.m[jcur], tile * (uint32_t)kBlocksPerTile + (e0 >> 5), stage);
                        
                    } else {
                        store_round_ragged(y + e0, stage, len - e0 < (uint32_t)kRound ? len - e0 : (uint32_t)kRound, lane);
                    }
                }
            }
        }
        cur = nxt;
        cb ^= 1u;
        t = tn;
    }
    if (lane == 0) asm volatile("cp.async.bulk.wait_group 0;" ::: "memory");
    if (status) atomicOr(ws.status, status);
}

// ------------------------------------------------------------------------------------------------ fused hop
//
// out = compress(decompress(in_c) (+) local), tile by tile, with no uncompressed intermediate in global memory: a
// warp decodes a round of the incoming tile straight onto the local operand's round (tensor copy, one round ahead;
// or a second compressed stream, decoded first), leaves the combined values in a stage, and encodes that stage like
// a round of the compressor: into a buffer, off to the round's slot by a bulk store.  The place kernel finishes the
// stream.  An uncompressed copy of the result, when asked for, leaves the stage by a tensor store.

// Out-of-line copies for the hop, whose kernel holds a decoder and an encoder: inlined, the compiler multiplied their
// code along the kernel's branches until instruction fetch bounded it (four times the size, 15 % slower).
template <int N, int MODE>
__device__ __noinline__ void decode_round_call(const uint32_t* blob, uint32_t padw, uint32_t L, uint32_t* pay_off, int32_t* code, float s,
                                               float* stage, int lane, const float* loc_stage)
{
    decode_round_n<N, MODE>(blob, padw, L, *pay_off, *code, s, stage, lane, loc_stage);
}
// the round by its width class (MODE as for expand_block); op: the reduce operation, for the general route
template <int MODE>
__device__ __forceinline__ void decode_round_classes(const uint32_t* blob, uint32_t padw, uint32_t L, uint32_t* pay_off, int32_t* code,
                                                     float s, float* stage, int lane, const float* loc_stage, uint32_t op)
{
    const int cls = round_class(L);
    if (cls == 8) decode_round_call<8, MODE>(blob, padw, L, pay_off, code, s, stage, lane, loc_stage);
    else if (cls == 16) decode_round_call<16, MODE>(blob, padw, L, pay_off, code, s, stage, lane, loc_stage);
    else decode_round_general(blob, padw, L, pay_off, code, s, stage, lane, loc_stage, op);
}
template <int N>
__device__ __noinline__ int encode_round_call(const char* row, uint32_t sw, float xprev, float r, bool active, uint32_t* buf, EncodeCarry* cy, int lane,
                                              uint32_t* status)
{
    // laid out like a tile's blob whose word 0 sits in front of the buffer: code-length bytes at words 1.., payload at word 9
    return encode_round_n<N>(row, sw, xprev, r, active, (uint32_t)lane, 32u, buf - 1, 0u, 1, 9u, (uint32_t)kRoundBufWords - 8u, *cy, lane, *status, [] {});
}

// Advances (pay_off, code) over round e of a tile without expanding it: the blocks' sizes from their code lengths,
// their sums of deltas from population counts of their planes.  Lets a warp start in the middle of a tile.
__device__ __noinline__ void skip_round(const uint32_t* blob, uint32_t padw, uint32_t L, uint32_t* pay_off, int32_t* code, int lane)
{
    const uint32_t nw = L ? L + 1u : 0u;
    const uint32_t incl = warp_incl_scan(nw, lane);
    const uint32_t* pay = blob + 1 + padw + *pay_off + (incl - nw);
    const uint32_t sign = L ? pay[0] : 0u;
    int32_t total = 0;
    for (uint32_t k = 0; k < L; ++k) {
        const uint32_t w = pay[1 + k];
        total += (__popc(w) - 2 * __popc(w & sign)) << k;
    }
    *pay_off += __shfl_sync(kFull, incl, 31);
    *code += (int32_t)__reduce_add_sync(kFull, total);
}

__device__ __forceinline__ uint32_t cj_begin_of(const JobBatch& jb, int j) { return jb.job[j].tile_begin; }

struct alignas(1024) HopWarpShared {
    float loc[2][kRound];                  // the operand's rounds, replaced in place by the combined values and then by
                                           // the encoded round; 1024-byte boundaries
    alignas(16) uint32_t blob[kDecBlobWords];
    alignas(8) unsigned long long bar_loc[2], bar_blob;
};
static_assert(sizeof(HopWarpShared) == 13 * 1024, "a warp's share of the shared memory");

// The owner's copy as the dequantised value float(q(y)) * s: `count` elements of the stage, coalesced.
__device__ __noinline__ void store_round_dequantised(float* __restrict__ y, const float* stage, uint32_t count, float r, float s, int lane)
{
#pragma unroll 4
    for (int k = 0; k < 32; ++k) {
        const uint32_t e = 32u * k + (uint32_t)lane;
        const float v = *reinterpret_cast<const float*>(reinterpret_cast<const char*>(stage) + stage_chunk_byte(k, (uint32_t)lane >> 2) + 4 * (lane & 3));
        if (e < count) y[e] = __fmul_rn(__int2float_rn(__float2int_rn(__fmul_rn(v, r))), s);
    }
}

// maps: tensor map of job j's uncompressed operand at [j] and, in launches of at most kMaxJobs / 2 jobs, of its
// uncompressed result at [kMaxJobs / 2 + j] (a second array of maps made the parameters 22 KB and the launch 1.6 us
// slower; launches with more jobs write such results with plain stores).
template <bool C2, bool Y, bool SPLIT>
__global__ void __launch_bounds__(kCodecThreads, 4) hop_tiles_kernel(const __grid_constant__ JobBatch jb, const __grid_constant__ TileMaps maps,
                                                                     Workspace ws, uint32_t split_shift_arg)
{
    const uint32_t split_shift = SPLIT ? split_shift_arg : 0u;   // SPLIT false: whole tiles only, known when the kernel is compiled
    // split_shift 0: a warp's unit of work is a tile; 1: two rounds; 2: a round (small launches: more warps at work, and
    // none of them walks four rounds in a row)
    pdl_enter();
    extern __shared__ __align__(16) unsigned char smem_raw[];
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    HopWarpShared& sh = reinterpret_cast<HopWarpShared*>(smem_raw + ((1024u - (smem_u32(smem_raw) & 1023u)) & 1023u))[warp];
    uint32_t status = 0;
    if (lane == 0) {
        mbar_init(&sh.bar_loc[0], 1); mbar_init(&sh.bar_loc[1], 1);
        mbar_init(&sh.bar_blob, 1);
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    __syncwarp();
    uint32_t lfill0 = 0, lfill1 = 0, bfill = 0;   // completed copies per buffer (phase parities)
    bool lbulk0 = false, lbulk1 = false;

    // the job of the tile looked up last, with its streams' headers
    int cj = -1;
    uint32_t cj_begin = 0, cj_count = 0;
    StreamInfo h1, h2;
    h1.ok = h2.ok = false; h1.n = h2.n = 0; h1.nT = h2.nT = 0; h1.s = h2.s = 1.0f; h1.eb_abs = h2.eb_abs = 0.0f;
    bool job_ok = false;
    auto enter_job = [&](uint32_t t) {
        if (t - cj_begin >= cj_count) {
            cj = find_job(jb, t);
            const Job& q = jb.job[cj];
            cj_begin = q.tile_begin;
            cj_count = (cj + 1 < jb.count ? jb.job[cj + 1].tile_begin : jb.total_tiles) - cj_begin;
            h1 = read_header(q.in_c, q.in_cap);
            job_ok = h1.ok && h1.n == q.n;
            if (C2 && q.in_c2) {
                h2 = read_header(q.in_c2, q.in2_cap);
                job_ok = job_ok && h2.ok && h2.n == q.n && __float_as_uint(h2.s) == __float_as_uint(h1.s);
            }
        }
    };
    // a tile's blob out of one of the job's streams, from the index alone (ptr = nullptr, words = ~0: damaged index)
    auto blob_of = [&](const uint32_t* in, unsigned long long cap, uint32_t nT, uint32_t tile) {
        BlobRef br;
        br.ptr = nullptr; br.words = 0xFFFFFFFFu; br.staged = false;
        const uint32_t* idx = in + kHeaderWords;
        const uint32_t w_end = ldg_u32(idx + tile), w_beg = tile ? ldg_u32(idx + tile - 1) : 0u;
        const unsigned long long blob0 = (unsigned long long)kHeaderWords + nT;
        if (w_end <= w_beg || (blob0 + w_end) * 4ull > cap) return br;
        br.ptr = in + blob0 + w_beg;
        br.words = w_end - w_beg;
        return br;
    };
    // the incoming blob of tile t of the launch; its cover is requested into the blob buffer when it fits
    auto request_blob = [&](uint32_t t) {
        BlobRef br;
        br.ptr = nullptr; br.words = 0; br.staged = false;
        if (t >= jb.total_tiles) return br;
        enter_job(t);
        const Job& q = jb.job[cj];
        const uint32_t tile = t - cj_begin;
        if (!job_ok || q.n == 0 || tile >= h1.nT) return br;
        br = blob_of(q.in_c, q.in_cap, h1.nT, tile);
        if (!br.ptr) return br;
        const uintptr_t a_end = ((uintptr_t)(br.ptr + br.words) + 15) & ~(uintptr_t)15;
        if (a_end - (uintptr_t)q.in_c <= (uintptr_t)q.in_cap) {   // the copies may read up to the boundary behind the blob
            if (lane == 0) window_request(br, 0, sh.blob, &sh.bar_blob);
            br.staged = true;
        }
        return br;
    };
    // round rd of the uncompressed operand of tile `tile` of the current job into operand stage `buf`
    auto request_loc = [&](int job_index, uint32_t tile, uint32_t rd, uint32_t buf) {
        bool bulk = false;
        const Job& q = jb.job[job_index];
        if (q.x) {
            const unsigned long long start = (unsigned long long)tile * kTile;
            const uint32_t len = (uint32_t)((q.n - start < (unsigned long long)kTile) ? (q.n - start) : kTile);
            const uint32_t e0 = rd * (uint32_t)kRound;
            if (e0 < len) {
                if ((((uintptr_t)q.x) & 15u) == 0 && e0 + (uint32_t)kRound <= len) {
                    if (lane == 0) tensor_load_round(sh.loc[buf], &sh.bar_loc[buf], &maps.m[job_index], tile * (uint32_t)kBlocksPerTile + (e0 >> 5));
                    bulk = true;
                } else load_round_ragged(sh.loc[buf], q.x + start, e0, len, lane);
            }
        }
        if (buf) lbulk1 = bulk; else lbulk0 = bulk;
    };
    auto arrive_loc = [&](uint32_t buf) {
        if (buf ? lbulk1 : lbulk0) {
            if (!mbar_wait(&sh.bar_loc[buf], (buf ? lfill1 : lfill0) & 1u)) status |= kStTimeout;
            if (buf) ++lfill1; else ++lfill0;
        }
        if (buf) lbulk1 = false; else lbulk0 = false;
        __syncwarp();
    };

    const uint32_t stride = gridDim.x * (uint32_t)kCodecWarps;
    const uint32_t total_units = jb.total_tiles << split_shift, rd_mask = (1u << split_shift) - 1u;
    uint32_t un = blockIdx.x * (uint32_t)kCodecWarps + (uint32_t)warp;   // unit: tile un >> split_shift, from round un & rd_mask on
    uint32_t pl = 0;   // operand stage in turn
    BlobRef cur = request_blob(un < total_units ? un >> split_shift : 0xFFFFFFFFu);
    if (un < total_units && job_ok && jb.job[cj].n) request_loc(cj, (un >> split_shift) - cj_begin, (un & rd_mask) * (4u >> split_shift), 0);
    EncodeCarry cy;
    cy.pay_used = 0; cy.wide = false;

    while (un < total_units) {
        const uint32_t t = un >> split_shift, rd_first = (un & rd_mask) * (4u >> split_shift);
        // the current tile's facts, before the look-up of the next tile moves on to another job
        enter_job(t);
        const int jcur = cj;
        const Job& job = jb.job[jcur];
        const uint32_t tile = t - cj_begin;
        const StreamInfo hc1 = h1, hc2 = h2;
        const bool ok = job_ok;
        const unsigned long long n = job.n;
        const float s = hc1.s, r = __fdiv_rn(1.0f, hc1.s);
        const unsigned long long start = (unsigned long long)tile * kTile;
        const uint32_t len = (ok && n) ? (uint32_t)((n - start < (unsigned long long)kTile) ? (n - start) : kTile) : 0u;
        const uint32_t nb = (len + kBlock - 1) / kBlock, padw = (nb + 3) >> 2, rounds = (nb + 31) >> 5;
        const uint32_t op = (job.flags >> 1) & 3u;
        const bool summing = op == 0u || op == 3u, deq = (job.flags & 1u) != 0;
        if (!ok) status |= kStBadStream;

        const uint32_t unn = (un + stride < un || un + stride >= total_units) ? 0xFFFFFFFFu : un + stride;
        const uint32_t tn = unn == 0xFFFFFFFFu ? 0xFFFFFFFFu : unn >> split_shift, nrd = (unn & rd_mask) * (4u >> split_shift);
        const uint32_t rd_end = rd_first + (4u >> split_shift);
        const uint32_t rd_stop = rd_first >= rounds ? rd_first : (rd_end < rounds ? rd_end : rounds);   // rounds [rd_first, rd_stop)
        if (cur.staged) {
            if (!mbar_wait(&sh.bar_blob, bfill & 1u)) status |= kStTimeout;
            ++bfill;
        }

        // what the two blobs say
        const uint32_t* blob1 = nullptr;
        const uint32_t* blob2 = nullptr;
        BlobWindow win;   // over the incoming blob
        win.base = nullptr; win.end = 0;
        int mode1 = 0, mode2 = 1;
        if (len) {
            if (cur.ptr) {
                win.base = cur.ptr; win.end = cur.words;
                if (cur.staged) win = window_at(cur, 0, sh.blob);
                blob1 = win.base;
                mode1 = describe_blob(blob1, cur.words, nb, lane);   // the head (at most 33 words) is in every first window
            }
            if (C2 && job.in_c2) {
                const BlobRef b2 = blob_of(job.in_c2, job.in2_cap, hc2.nT, tile);
                blob2 = b2.ptr;
                mode2 = b2.ptr ? describe_blob(b2.ptr, b2.words, nb, lane) : 0;
            }
            if (mode1 == 0 || mode2 == 0) status |= kStBadStream;
        }
        const bool good = len != 0 && mode1 != 0 && mode2 != 0;

        uint32_t pay1 = 0, pay2 = 0;
        int32_t code1 = good ? (int32_t)blob1[0] : 0, code2 = (C2 && good && blob2) ? (int32_t)blob2[0] : 0;
        const uint32_t lp1 = good ? lane_code_lengths(blob1, nb, lane) : 0u, lp2 = (C2 && good && blob2) ? lane_code_lengths(blob2, nb, lane) : 0u;
        // moves the window over the incoming blob to round e's first word when the round reaches past its end
        auto reach = [&](uint32_t e) {
            const uint32_t L = (lp1 >> (8u * e)) & 0xFFu;
            const uint32_t first = 1u + padw + pay1;
            if (win.end < cur.words && first + __reduce_add_sync(kFull, L ? L + 1u : 0u) > win.end) {
                __syncwarp();   // every lane is done with the window as it is
                if (lane == 0) window_request(cur, first, sh.blob, &sh.bar_blob);
                if (!mbar_wait(&sh.bar_blob, bfill & 1u)) status |= kStTimeout;
                ++bfill;
                win = window_at(cur, first, sh.blob);
                blob1 = win.base;
            }
            return L;
        };
        float carry_y = 0.0f;
        // The next tile's blob goes into the one blob buffer as soon as this tile's last round is decoded; that look-up
        // moves the job on, so the next tile's facts are kept from there.
        BlobRef nxt;
        nxt.ptr = nullptr; nxt.words = 0; nxt.staged = false;
        bool next_has_operand = false, next_known = false;
        int njob = 0;
        uint32_t ntile = 0;
        auto look_ahead = [&]() {
            __syncwarp();   // every lane is done with the blob buffer
            nxt = request_blob(tn);
            next_has_operand = tn < jb.total_tiles && job_ok && jb.job[cj].n != 0;
            njob = cj;
            ntile = tn - cj_begin;
            next_known = true;
        };
        if (rd_first >= rd_stop || !good) look_ahead();
        if (good && rd_first != 0 && rd_first < rd_stop) {
            // a unit that starts inside its tile: sizes and codes of the rounds in front, and the value in front of it
            for (uint32_t e = 0; e < rd_first; ++e) {
                const uint32_t Le = reach(e);
                skip_round(blob1, padw, Le, &pay1, &code1, lane);
                if (C2 && blob2) skip_round(blob2, padw, (lp2 >> (8u * e)) & 0xFFu, &pay2, &code2, lane);
            }
            const float xa = __fmul_rn(__int2float_rn(code1), s);
            const float xb = (C2 && blob2) ? __fmul_rn(__int2float_rn(code2), s) : __ldg(job.x + start + rd_first * (uint32_t)kRound - 1u);
            carry_y = combine(op, xa, xb);
        }
        for (uint32_t rd = rd_first; rd < rd_stop; ++rd) {
            // The other operand stage holds the round before, encoded in place and handed to the copy engine: the next
            // operand round is asked into it once the engine is through with it, which by the end of this round's decoding it
            // mostly is.
            auto release_other = [&]() {
                if (lane == 0) asm volatile("cp.async.bulk.wait_group.read 0;" ::: "memory");
                __syncwarp();
            };
            float* loc = sh.loc[pl];
            const uint32_t u = 4u * t + rd;
            if (!good) {
                release_other();
                if (rd + 1 < rd_stop) request_loc(jcur, tile, rd + 1, pl ^ 1u);
                else if (next_has_operand) request_loc(njob, ntile, nrd, pl ^ 1u);
                else { if (pl) lbulk0 = false; else lbulk1 = false; }
                arrive_loc(pl);
                if (lane == 0) ws.round_words[u] = 0;
            } else {
                arrive_loc(pl);
                if (C2 && blob2) {   // the operand is compressed too: its round goes where an uncompressed one would be
                    const uint32_t L2 = (lp2 >> (8u * rd)) & 0xFFu;
                    if (mode2 == 1) decode_round_classes<0>(blob2, padw, L2, &pay2, &code2, s, loc, lane, nullptr, 0u);
                    else decode_round_general(blob2, padw, L2, &pay2, &code2, s, loc, lane, nullptr, 0u);
                    __syncwarp();
                }
                const uint32_t L1 = reach(rd);
                if (mode1 == 1 && summing) decode_round_classes<1>(blob1, padw, L1, &pay1, &code1, s, loc, lane, loc, op);
                else decode_round_general(blob1, padw, L1, &pay1, &code1, s, loc, lane, loc, op);
                release_other();
                if (rd + 1 < rd_stop) request_loc(jcur, tile, rd + 1, pl ^ 1u);
                else {   // the blob is decoded: the next unit's may come, and its first operand round
                    look_ahead();
                    if (next_has_operand) request_loc(njob, ntile, nrd, pl ^ 1u);
                    else { if (pl) lbulk0 = false; else lbulk1 = false; }
                }
                __syncwarp();   // the stage's rows, written by all lanes, are visible
                const float* ys = loc;
                const char* row = reinterpret_cast<const char*>(ys) + 128 * lane;
                const uint32_t sw = ((uint32_t)lane & 7u) << 4;
                const float y0 = ys[0];
                const float xprev = lane ? read_last_of_row(ys, (uint32_t)lane - 1u) : (rd ? carry_y : y0);   // carry_y: the value in front of the round
                carry_y = read_last_of_row(ys, 31);
                const uint32_t e0 = rd * (uint32_t)kRound;
                uint32_t* slot = ws.slots + (size_t)u * kRoundSlotWords;
                if (Y && job.y) {   // an uncompressed copy of the result leaves the stage before the encoder writes over it
                    const uint32_t count = len - e0 < (uint32_t)kRound ? len - e0 : (uint32_t)kRound;
                    if (deq) store_round_dequantised(job.y + start + e0, ys, count, r, s, lane);
                    else if (jb.count <= kMaxJobs / 2 && (((uintptr_t)job.y) & 15u) == 0 && count == (uint32_t)kRound) {
                        if (lane == 0) {
                            tensor_store_round(&maps.m[kMaxJobs / 2 + jcur], tile * (uint32_t)kBlocksPerTile + (e0 >> 5), ys);
                            asm volatile("cp.async.bulk.wait_group.read 0;" ::: "memory");
                        }
                    } else store_round_ragged(job.y + start + e0, ys, count, lane);
                    __syncwarp();
                }
                uint32_t* buf = reinterpret_cast<uint32_t*>(loc);   // in place: a round's code never outgrows its 4 KiB
                cy.pay_used = 0;
                const uint32_t bi = 32u * rd + (uint32_t)lane;
                int rc = 3;
                if (!cy.wide) rc = encode_round_call<8>(row, sw, xprev, r, bi < nb, buf, &cy, lane, &status);
                if (rc == 3) rc = encode_round_call<16>(row, sw, xprev, r, bi < nb, buf, &cy, lane, &status);
                const uint32_t gslot = (cj_begin_of(jb, jcur) >> 5) + (uint32_t)jcur + (tile >> 5);
                if (rc == 0) {
                    __syncwarp();   // the buffer's words, written by all lanes, are visible to lane 0's store
                    if (lane == 0) {
                        const uint32_t bytes = (32u + 4u * cy.pay_used + 15u) & ~15u;
                        asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
                        asm volatile("cp.async.bulk.global.shared::cta.bulk_group [%0], [%1], %2;" ::"l"(slot), "r"(smem_u32(buf)), "r"(bytes) : "memory");
                        asm volatile("cp.async.bulk.commit_group;" ::: "memory");
                        ws.round_words[u] = cy.pay_used;
                        atomicAdd(ws.group_acc + gslot, (unsigned long long)cy.pay_used);
                        // exact while |y r| < 2^22; larger codes take the general route
                        if (rd == 0) ws.outliers[t] = (int32_t)(__float_as_uint(__fadd_rn(__fmul_rn(y0, r), kRoundMagic)) - kRoundMagicBits);
                    }
                } else {
                    status |= encode_round_general_staged(ys, xprev, bi < nb, rd, r, slot, ws.round_words + u, ws.outliers + t, ws.group_acc + gslot, lane);
                }
            }
            pl ^= 1u;
        }
        if (rd_first >= rd_stop && next_has_operand) {
            if (lane == 0) asm volatile("cp.async.bulk.wait_group.read 0;" ::: "memory");   // the stage may still be on its way out
            __syncwarp();
            request_loc(njob, ntile, nrd, pl);
        }
        // rounds the tile does not have
        if ((uint32_t)lane >= rd_first && (uint32_t)lane < rd_end && (uint32_t)lane >= rounds) ws.round_words[4u * t + (uint32_t)lane] = 0;
        (void)next_known;
        cur = nxt;
        un = unn;
    }
    if (lane == 0) asm volatile("cp.async.bulk.wait_group 0;" ::: "memory");
    if (status) atomicOr(ws.status, status);
}

#include "zccl_codec_f64.cuh"
#include "zccl_codec_tiled.cuh"

// Per-device launch set-up (shared-memory attribute, resident CTAs per SM), done once per device under a lock.
constexpr int kMaxDevices = 64;
constexpr size_t kEncSmemBytes = sizeof(EncWarpShared) * kCodecWarps + 1024;   // + room to reach a 1024-byte boundary
constexpr size_t kRoundSmemBytes = sizeof(RoundWarpShared) * kCodecWarps + 1024;
constexpr size_t kDecSmemBytes = sizeof(DecWarpShared) * kCodecWarps + 1024;
constexpr size_t kHopSmemBytes = sizeof(HopWarpShared) * kCodecWarps + 1024;
constexpr size_t kRound64SmemBytes = sizeof(RoundWarpShared64) * kCodecWarps + 1024;
constexpr size_t kDec64SmemBytes = sizeof(DecWarpShared64) * kCodecWarps + 1024;
struct DeviceSetup {
    bool ready = false;
    int enc_ctas = 1, round_ctas = 1, dec_ctas = 1, hop_ctas = 1, round64_ctas = 1, dec64_ctas = 1, round_tiled_ctas = 1, dec_tiled_ctas = 1;
};
DeviceSetup g_dev[kMaxDevices];
std::mutex g_dev_mu;
using EncodeTiledFn = CUresult (*)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*, const cuuint64_t*, const cuuint32_t*,
                                   const cuuint32_t*, CUtensorMapInterleave, CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);
EncodeTiledFn g_encode_tiled = nullptr;   // the driver's cuTensorMapEncodeTiled, looked up through the runtime

// The eight forms of the hop kernel (see hop_tiles_kernel's template parameters), by index 4 C2 + 2 Y + SPLIT.
using HopLaunch = cudaError_t (*)(dim3, cudaStream_t, const JobBatch&, const TileMaps&, const Workspace&, uint32_t);
template <bool C2, bool Y, bool SPLIT>
cudaError_t hop_launch(dim3 grid, cudaStream_t st, const JobBatch& jb, const TileMaps& maps, const Workspace& ws, uint32_t split_shift)
{
    return launch_k(hop_tiles_kernel<C2, Y, SPLIT>, grid, dim3(kCodecThreads), kHopSmemBytes, st, jb, maps, ws, split_shift);
}
inline HopLaunch hop_form(bool c2, bool y, bool split)
{
    static const HopLaunch forms[8] = {hop_launch<false, false, false>, hop_launch<false, false, true>, hop_launch<false, true, false>,
                                       hop_launch<false, true, true>,   hop_launch<true, false, false>, hop_launch<true, false, true>,
                                       hop_launch<true, true, false>,   hop_launch<true, true, true>};
    return forms[(c2 ? 4 : 0) + (y ? 2 : 0) + (split ? 1 : 0)];
}
template <bool C2, bool Y, bool SPLIT>
cudaError_t hop_smem_attr() { return cudaFuncSetAttribute(hop_tiles_kernel<C2, Y, SPLIT>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)kHopSmemBytes); }

cudaError_t device_setup(const DeviceSetup** out)
{
    int dev = 0;
    cudaError_t e = cudaGetDevice(&dev);
    if (e != cudaSuccess) return e;
    if (dev < 0 || dev >= kMaxDevices) return cudaErrorInvalidDevice;
    std::lock_guard<std::mutex> lock(g_dev_mu);
    if (!g_encode_tiled) {
        void* fn = nullptr;
        cudaDriverEntryPointQueryResult q;
        e = cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &fn, cudaEnableDefault, &q);
        if (e != cudaSuccess) return e;
        if (q != cudaDriverEntryPointSuccess || !fn) return cudaErrorNotSupported;
        g_encode_tiled = reinterpret_cast<EncodeTiledFn>(fn);
    }
    DeviceSetup& d = g_dev[dev];
    if (!d.ready) {
        e = cudaFuncSetAttribute(enc_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)kEncSmemBytes);
        if (e != cudaSuccess) return e;
        int a = 0;
        e = cudaOccupancyMaxActiveBlocksPerMultiprocessor(&a, enc_kernel, kCodecThreads, kEncSmemBytes);
        if (e != cudaSuccess) return e;
        d.enc_ctas = a > 0 ? a : 1;
        e = cudaFuncSetAttribute(encode_rounds_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)kRoundSmemBytes);
        if (e != cudaSuccess) return e;
        e = cudaOccupancyMaxActiveBlocksPerMultiprocessor(&a, encode_rounds_kernel, kCodecThreads, kRoundSmemBytes);
        if (e != cudaSuccess) return e;
        d.round_ctas = a > 0 ? a : 1;
        e = cudaFuncSetAttribute(decode_tiles_kernel<kMaxJobs>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)kDecSmemBytes);
        if (e != cudaSuccess) return e;
        e = cudaFuncSetAttribute(decode_tiles_kernel<kMaxDecodeJobs>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)kDecSmemBytes);
        if (e != cudaSuccess) return e;
        e = cudaOccupancyMaxActiveBlocksPerMultiprocessor(&a, decode_tiles_kernel<kMaxJobs>, kCodecThreads, kDecSmemBytes);
        if (e != cudaSuccess) return e;
        d.dec_ctas = a > 0 ? a : 1;
        e = cudaFuncSetAttribute(place_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)kPlaceSmemBytes);
        if (e != cudaSuccess) return e;
        e = hop_smem_attr<false, false, false>();
        if (e == cudaSuccess) e = hop_smem_attr<false, false, true>();
        if (e == cudaSuccess) e = hop_smem_attr<false, true, false>();
        if (e == cudaSuccess) e = hop_smem_attr<false, true, true>();
        if (e == cudaSuccess) e = hop_smem_attr<true, false, false>();
        if (e == cudaSuccess) e = hop_smem_attr<true, false, true>();
        if (e == cudaSuccess) e = hop_smem_attr<true, true, false>();
        if (e == cudaSuccess) e = hop_smem_attr<true, true, true>();
        if (e != cudaSuccess) return e;
        e = cudaOccupancyMaxActiveBlocksPerMultiprocessor(&a, hop_tiles_kernel<true, true, true>, kCodecThreads, kHopSmemBytes);
        if (e != cudaSuccess) return e;
        d.hop_ctas = a > 0 ? a : 1;
        e = cudaFuncSetAttribute(encode_rounds_f64_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)kRound64SmemBytes);
        if (e != cudaSuccess) return e;
        e = cudaOccupancyMaxActiveBlocksPerMultiprocessor(&a, encode_rounds_f64_kernel, kCodecThreads, kRound64SmemBytes);
        if (e != cudaSuccess) return e;
        d.round64_ctas = a > 0 ? a : 1;
        e = cudaFuncSetAttribute(decode_tiles_f64_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)kDec64SmemBytes);
        if (e != cudaSuccess) return e;
        e = cudaOccupancyMaxActiveBlocksPerMultiprocessor(&a, decode_tiles_f64_kernel, kCodecThreads, kDec64SmemBytes);
        if (e != cudaSuccess) return e;
        d.dec64_ctas = a > 0 ? a : 1;
        e = cudaFuncSetAttribute(encode_rounds_tiled_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)kRoundSmemBytes);
        if (e != cudaSuccess) return e;
        e = cudaOccupancyMaxActiveBlocksPerMultiprocessor(&a, encode_rounds_tiled_kernel, kCodecThreads, kRoundSmemBytes);
        if (e != cudaSuccess) return e;
        d.round_tiled_ctas = a > 0 ? a : 1;
        e = cudaFuncSetAttribute(decode_tiles_tiled_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)kDecSmemBytes);
        if (e != cudaSuccess) return e;
        e = cudaOccupancyMaxActiveBlocksPerMultiprocessor(&a, decode_tiles_tiled_kernel, kCodecThreads, kDecSmemBytes);
        if (e != cudaSuccess) return e;
        d.dec_tiled_ctas = a > 0 ? a : 1;
        d.ready = true;
    }
    *out = &d;
    return cudaSuccess;
}

// The array x of n floats as rows of 32 floats, copied in tiles of 32 rows with the 128-byte swizzle.  Arrays that
// do not start on a 16-byte boundary or have no full row get no map (the kernels load them element by element).
cudaError_t make_row_map(CUtensorMap* map, const float* x, unsigned long long n)
{
    if ((((uintptr_t)x) & 15u) != 0 || n < (unsigned long long)kBlock) return cudaSuccess;
    const cuuint64_t dims[2] = {(cuuint64_t)kBlock, (cuuint64_t)(n / kBlock)};
    const cuuint64_t strides[1] = {(cuuint64_t)kBlock * sizeof(float)};
    const cuuint32_t box[2] = {(cuuint32_t)kBlock, 32u};
    const cuuint32_t estr[2] = {1u, 1u};
    const CUresult r = g_encode_tiled(map, CU_TENSOR_MAP_DATA_TYPE_FLOAT32, 2, const_cast<float*>(x), dims, strides, box, estr,
                                      CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_128B,
                                      CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
    return r == CUDA_SUCCESS ? cudaSuccess : cudaErrorInvalidValue;
}

// The array x of n doubles as rows of 16 doubles, copied in tiles of 64 rows with the 128-byte swizzle.
cudaError_t make_row_map_f64(CUtensorMap* map, const double* x, unsigned long long n)
{
    if ((((uintptr_t)x) & 15u) != 0 || n < 16ull) return cudaSuccess;
    const cuuint64_t dims[2] = {16u, (cuuint64_t)(n / 16ull)};
    const cuuint64_t strides[1] = {16u * sizeof(double)};
    const cuuint32_t box[2] = {16u, (cuuint32_t)kRowsPerRound64};
    const cuuint32_t estr[2] = {1u, 1u};
    const CUresult r = g_encode_tiled(map, CU_TENSOR_MAP_DATA_TYPE_FLOAT64, 2, const_cast<double*>(x), dims, strides, box, estr,
                                      CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_128B,
                                      CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
    return r == CUDA_SUCCESS ? cudaSuccess : cudaErrorInvalidValue;
}

}  // namespace

// one CTA of the place kernel per group of 32 tiles of every job
uint32_t group_table(const JobBatch& jb, GroupTable& gt)
{
    uint32_t groups = 0;
    for (int j = 0; j < jb.count; ++j) {
        gt.begin[j] = groups;
        const uint32_t tiles = (j + 1 < jb.count ? jb.job[j + 1].tile_begin : jb.total_tiles) - jb.job[j].tile_begin;
        groups += (tiles + 31u) / 32u;
    }
    for (int j = jb.count; j <= kMaxJobs; ++j) gt.begin[j] = groups;
    return groups;
}

cudaError_t launch_hop_lanes(const JobBatch& jb, const Workspace& ws, int sm_count, cudaStream_t st)
{
    const DeviceSetup* d = nullptr;
    cudaError_t e = device_setup(&d);
    if (e != cudaSuccess) return e;
    if (!ws.slots) return cudaErrorInvalidValue;
    thread_local TileMaps maps;   // 8 KiB: kept off the stack, one per calling thread
    memset(&maps, 0, sizeof(maps));
    for (int j = 0; j < jb.count; ++j) {
        if (jb.job[j].x && (e = make_row_map(&maps.m[j], jb.job[j].x, jb.job[j].n)) != cudaSuccess) return e;
        if (jb.count <= kMaxJobs / 2 && jb.job[j].y && (e = make_row_map(&maps.m[kMaxJobs / 2 + j], jb.job[j].y, jb.job[j].n)) != cudaSuccess)
            return e;
    }
    GroupTable gt;
    const uint32_t groups = group_table(jb, gt);
    const unsigned long long cap = (unsigned long long)sm_count * d->hop_ctas;
    // launches that would leave warps idle with a tile per warp (a ring's hops) hand out rounds instead
    const unsigned long long warps = cap * kCodecWarps;
    const uint32_t split_shift = 4ull * jb.total_tiles <= warps ? 2u : 2ull * jb.total_tiles <= warps ? 1u : 0u;
    const unsigned long long want = ((((unsigned long long)jb.total_tiles) << split_shift) + kCodecWarps - 1) / kCodecWarps;
    // the kernel comes in eight forms: with or without the code for a compressed second operand, for an uncompressed copy
    // of the result, and for units that start inside tiles, none of which the hop of a large chunk has
    bool c2 = false, y = false;
    for (int j = 0; j < jb.count; ++j) { c2 = c2 || jb.job[j].in_c2 != nullptr; y = y || jb.job[j].y != nullptr; }
    const dim3 grid((unsigned)(want < cap ? want : cap));
    e = hop_form(c2, y, split_shift != 0)(grid, st, jb, maps, ws, split_shift);
    if (e != cudaSuccess) return e;
    return launch_k(place_kernel, dim3(groups), dim3(kPlaceThreads), kPlaceSmemBytes, st, jb, gt, ws, Params{0.f, 1.f, 1.f, 1}, 0, 1, ParamsF64{0.0, 1.0, 1.0, 1});
}

template <int CAP>
static cudaError_t launch_decode_lanes_t(const JobBatchT<CAP>& jb, const Workspace& ws, int sm_count, cudaStream_t st)
{
    const DeviceSetup* d = nullptr;
    cudaError_t e = device_setup(&d);
    if (e != cudaSuccess) return e;
    thread_local TileMapsT<CAP> maps;   // kept off the stack, one per calling thread
    memset(&maps, 0, sizeof(maps));
    for (int j = 0; j < jb.count; ++j)
        if ((e = make_row_map(&maps.m[j], jb.job[j].y, jb.job[j].n)) != cudaSuccess) return e;
    const unsigned long long want = ((unsigned long long)jb.total_tiles + kCodecWarps - 1) / kCodecWarps;
    const unsigned long long cap = (unsigned long long)sm_count * d->dec_ctas;
    return launch_k(decode_tiles_kernel<CAP>, dim3((unsigned)(want < cap ? want : cap)), dim3(kCodecThreads), kDecSmemBytes, st, jb, maps, ws);
}
cudaError_t launch_decode_lanes(const JobBatch& jb, const Workspace& ws, int sm_count, cudaStream_t st)
{
    return launch_decode_lanes_t<kMaxJobs>(jb, ws, sm_count, st);
}
cudaError_t launch_decode_lanes_wide(const DecodeBatch& jb, const Workspace& ws, int sm_count, cudaStream_t st)
{
    return launch_decode_lanes_t<kMaxDecodeJobs>(jb, ws, sm_count, st);
}


cudaError_t launch_encode_lanes(const JobBatch& jb, const Workspace& ws, bool device_params, Params host_params, int sm_count,
                                cudaStream_t st)
{
    const DeviceSetup* d = nullptr;
    cudaError_t e = device_setup(&d);
    if (e != cudaSuccess) return e;
    TileMaps maps;
    memset(&maps, 0, sizeof(maps));
    for (int j = 0; j < jb.count; ++j)
        if ((e = make_row_map(&maps.m[j], jb.job[j].x, jb.job[j].n)) != cudaSuccess) return e;
    if (ws.slots && ws.skip_publish == 0xFFFFFFFFu) {
        // two steps: rounds into their slots, then one CTA per group of 32 tiles places them
        GroupTable gt;
        const uint32_t groups = group_table(jb, gt);
        const unsigned long long rounds = (unsigned long long)jb.total_tiles * kRoundsPerTile;
        const unsigned long long want_a = (rounds + kCodecWarps - 1) / kCodecWarps;
        const unsigned long long cap_a = (unsigned long long)sm_count * d->round_ctas;
        e = launch_k(encode_rounds_kernel, dim3((unsigned)(want_a < cap_a ? want_a : cap_a)), dim3(kCodecThreads), kRoundSmemBytes, st, jb, maps, ws,
                     host_params, device_params ? 1 : 0);
        if (e != cudaSuccess) return e;
        return launch_k(place_kernel, dim3(groups), dim3(kPlaceThreads), kPlaceSmemBytes, st, jb, gt, ws, host_params, device_params ? 1 : 0, 0, ParamsF64{0.0, 1.0, 1.0, 1});
    }
    const unsigned long long want = ((unsigned long long)jb.total_tiles + kCodecWarps - 1) / kCodecWarps;
    unsigned long long cap = (unsigned long long)sm_count * d->enc_ctas;
    const unsigned grid = (unsigned)(want < cap ? want : cap);
    return launch_k(enc_kernel, dim3(grid), dim3(kCodecThreads), kEncSmemBytes, st, jb, maps, ws, host_params, device_params ? 1 : 0);
}

// Binary64 input: rounds into their slots, then the placement (two launches).
cudaError_t launch_encode_f64_lanes(const double* x, unsigned long long n, ParamsF64 hp, bool device_params, uint32_t* out,
                                    unsigned long long out_cap, size_t* out_bytes, const Workspace& ws, int sm_count, cudaStream_t st)
{
    const DeviceSetup* d = nullptr;
    cudaError_t e = device_setup(&d);
    if (e != cudaSuccess) return e;
    if (!ws.slots) return cudaErrorInvalidValue;
    CUtensorMap map;
    memset(&map, 0, sizeof(map));
    const bool mapped = (((uintptr_t)x) & 15u) == 0 && n >= 16ull;
    if (mapped && (e = make_row_map_f64(&map, x, n)) != cudaSuccess) return e;
    const unsigned long long nT = (n + kTile - 1) / kTile;
    thread_local JobBatch jb;
    memset(&jb, 0, sizeof(jb));
    jb.count = 1;
    jb.total_tiles = (uint32_t)(nT ? nT : 1);
    jb.job[0].x = reinterpret_cast<const float*>(x);
    jb.job[0].out = out; jb.job[0].out_bytes = out_bytes; jb.job[0].n = n; jb.job[0].out_cap = out_cap;
    if (jb.total_tiles > ws.max_tiles) return cudaErrorInvalidValue;
    GroupTable gt;
    const uint32_t groups = group_table(jb, gt);
    const unsigned long long cap = (unsigned long long)sm_count * d->round64_ctas;
    const unsigned grid = (unsigned)(jb.total_tiles < cap ? jb.total_tiles : cap);
    e = launch_k(encode_rounds_f64_kernel, dim3(grid), dim3(kCodecThreads), kRound64SmemBytes, st, x, n, jb.total_tiles, map, mapped ? 1 : 0, ws,
                 hp, device_params ? 1 : 0);
    if (e != cudaSuccess) return e;
    return launch_k(place_kernel, dim3(groups), dim3(kPlaceThreads), kPlaceSmemBytes, st, jb, gt, ws, Params{0.f, 1.f, 1.f, 1}, device_params ? 1 : 0, 2,
                    hp);
}

cudaError_t launch_decode_f64_lanes(const uint32_t* in, unsigned long long cap_bytes, double* y, unsigned long long y_cap, const Workspace& ws,
                                    int sm_count, cudaStream_t st)
{
    const DeviceSetup* d = nullptr;
    cudaError_t e = device_setup(&d);
    if (e != cudaSuccess) return e;
    CUtensorMap map;
    memset(&map, 0, sizeof(map));
    const bool mapped = (((uintptr_t)y) & 15u) == 0 && y_cap >= 16ull;
    if (mapped && (e = make_row_map_f64(&map, y, y_cap)) != cudaSuccess) return e;
    const unsigned long long tiles = (y_cap + kTile - 1) / kTile;
    if (tiles >= 0xFFFFFFFFull) return cudaErrorInvalidValue;
    const unsigned long long want = (tiles + kCodecWarps - 1) / kCodecWarps;
    const unsigned long long cap = (unsigned long long)sm_count * d->dec64_ctas;
    return launch_k(decode_tiles_f64_kernel, dim3((unsigned)(want < cap ? (want ? want : 1) : cap)), dim3(kCodecThreads), kDec64SmemBytes, st, in,
                    cap_bytes, y, y_cap, (uint32_t)tiles, map, mapped ? 1 : 0, ws);
}

// Binary32 at another tile size on the tuned kernels: rounds into their slots, then the placement.  False when the
// context's slots do not cover the launch (the caller then takes the plain kernels).
bool tiled_lanes_fit(unsigned long long n, uint32_t T, const Workspace& ws)
{
    const unsigned long long tiles = (n + T - 1) / T, R = (T + kRound - 1) / kRound;
    return ws.slots && tiles * R <= 4ull * ws.max_tiles;   // one slot per round; first codes and group sums are laid out for tiles of 1024
}

cudaError_t launch_encode_tiled_lanes(const float* x, unsigned long long n, uint32_t T, Params hp, bool device_params, uint32_t* out,
                                      unsigned long long out_cap, size_t* out_bytes, const Workspace& ws, int sm_count, cudaStream_t st)
{
    const DeviceSetup* d = nullptr;
    cudaError_t e = device_setup(&d);
    if (e != cudaSuccess) return e;
    if (!tiled_lanes_fit(n, T, ws)) return cudaErrorInvalidValue;
    CUtensorMap map;
    memset(&map, 0, sizeof(map));
    const bool mapped = (((uintptr_t)x) & 15u) == 0 && n >= (unsigned long long)kBlock;
    if (mapped && (e = make_row_map(&map, x, n)) != cudaSuccess) return e;
    TiledShape sp;
    sp.T = T; sp.R = (T + kRound - 1) / kRound; sp.lw_full = (T / kBlock + 3) / 4;
    const unsigned long long nT = (n + T - 1) / T;
    const uint32_t tiles = (uint32_t)(nT ? nT : 1);
    const unsigned long long rounds = (unsigned long long)tiles * sp.R;
    const unsigned long long want = (rounds + kCodecWarps - 1) / kCodecWarps;
    const unsigned long long cap = (unsigned long long)sm_count * d->round_tiled_ctas;
    e = launch_k(encode_rounds_tiled_kernel, dim3((unsigned)(want < cap ? want : cap)), dim3(kCodecThreads), kRoundSmemBytes, st, x, n, sp, tiles, map,
                 mapped ? 1 : 0, ws, hp, device_params ? 1 : 0);
    if (e != cudaSuccess) return e;
    return launch_k(place_tiled_kernel, dim3((tiles + 31u) / 32u), dim3(kPlaceThreads), 0, st, out, out_cap, out_bytes, n, sp, tiles, ws, hp,
                    device_params ? 1 : 0);
}

cudaError_t launch_decode_tiled_lanes(const uint32_t* in, unsigned long long cap_bytes, uint32_t T, float* y, unsigned long long y_cap,
                                      const Workspace& ws, int sm_count, cudaStream_t st)
{
    const DeviceSetup* d = nullptr;
    cudaError_t e = device_setup(&d);
    if (e != cudaSuccess) return e;
    CUtensorMap map;
    memset(&map, 0, sizeof(map));
    const bool mapped = (((uintptr_t)y) & 15u) == 0 && y_cap >= (unsigned long long)kBlock;
    if (mapped && (e = make_row_map(&map, y, y_cap)) != cudaSuccess) return e;
    TiledShape sp;
    sp.T = T; sp.R = (T + kRound - 1) / kRound; sp.lw_full = (T / kBlock + 3) / 4;
    const unsigned long long tiles = (y_cap + T - 1) / T;
    if (tiles >= 0xFFFFFFFFull) return cudaErrorInvalidValue;
    const unsigned long long want = (tiles + kCodecWarps - 1) / kCodecWarps;
    const unsigned long long cap = (unsigned long long)sm_count * d->dec_tiled_ctas;
    return launch_k(decode_tiles_tiled_kernel, dim3((unsigned)(want < cap ? (want ? want : 1) : cap)), dim3(kCodecThreads), kDecSmemBytes, st, in,
                    cap_bytes, sp, y, y_cap, (uint32_t)tiles, map, mapped ? 1 : 0, ws);
}

}  // namespace zccl
