// The binary32 format at other tile sizes (a multiple of 32 elements between 1024 and 8192; Section 3.5.2 cuts the
// data into chunks of 5120 points) on the lane-per-block decomposition: included by zccl_codec.cu inside its unnamed
// namespace.  A tile of T elements has R = ceil(T / 1024) rounds, the last one possibly partial; rounds are the unit
// of work of the encoder (round g of the launch = round g mod R of tile g / R), tiles that of the placement and of
// the decoder.  One array per launch.  The round encoder, the round decoder, the slots and the blob windows are
// those of the 4096-element kernels; what is new here is only the walk over rounds and tiles.

struct TiledShape {
    uint32_t T;        // elements per tile
    uint32_t R;        // rounds per tile
    uint32_t lw_full;  // code-length words of a full tile: ceil(T / 32 / 4)
};

__device__ __forceinline__ uint32_t tiled_len(unsigned long long n, unsigned long long t, uint32_t T)
{
    const unsigned long long left = n - t * T;
    return (uint32_t)(left < (unsigned long long)T ? left : (unsigned long long)T);
}

// Step 1 of a compression: every warp takes rounds g = warp number, + warps of the grid, ...; a full round of an array
// on a 16-byte boundary comes in by one tensor copy, other rounds by plain loads; the round is encoded in place and
// leaves by one bulk store to slot g (or takes the general route straight from global memory).
__global__ void __launch_bounds__(kCodecThreads, 4) encode_rounds_tiled_kernel(const float* __restrict__ x, unsigned long long n, TiledShape sp,
                                                                               uint32_t tiles, const __grid_constant__ CUtensorMap map, int mapped,
                                                                               Workspace ws, Params hp, int use_dev_params)
{
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
    const unsigned long long rounds = (unsigned long long)tiles * sp.R;
    const unsigned long long stride = (unsigned long long)gridDim.x * kCodecWarps;
    const uint32_t sw = ((uint32_t)lane & 7u) << 4;

    struct At { unsigned long long t; uint32_t rd, len; };
    auto at = [&](unsigned long long g) {
        At a;
        a.t = g / sp.R;
        a.rd = (uint32_t)(g - a.t * sp.R);
        a.len = (g < rounds && prm.valid && n) ? tiled_len(n, a.t, sp.T) : 0u;
        return a;
    };
    // Asks for round g into stage st; completes one phase of the stage's mbarrier whatever there is to bring.
    auto request = [&](unsigned long long g, uint32_t st) {
        const At a = at(g);
        const uint32_t e0 = a.rd * (uint32_t)kRound;
        if (e0 < a.len) {
            const float* xt = x + a.t * sp.T;
            if (mapped && e0 + (uint32_t)kRound <= a.len) {
                if (lane == 0) {
                    mbar_expect_tx(&sh.bar[st], kRound * 4 + (a.rd ? 16u : 0u));
                    asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
                    asm volatile("cp.async.bulk.tensor.2d.shared::cluster.global.tile.mbarrier::complete_tx::bytes [%0], [%1, {%2, %3}], [%4];"
                                 ::"r"(smem_u32(sh.stage[st])), "l"(&map), "r"(0), "r"((int)((a.t * sp.T + e0) >> 5)), "r"(smem_u32(&sh.bar[st]))
                                 : "memory");
                    if (a.rd)
                        asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], 16, [%2];"
                                     ::"r"(smem_u32(sh.front[st])), "l"(xt + e0 - 4), "r"(smem_u32(&sh.bar[st])) : "memory");
                }
                return;
            }
            load_round_ragged(sh.stage[st], xt, e0, a.len, lane);
            if (lane == 0 && a.rd) sh.front[st][3] = __ldg(xt + e0 - 1u);
            __syncwarp();
        }
        if (lane == 0) mbar_arrive(&sh.bar[st]);
    };

    unsigned long long g = (unsigned long long)blockIdx.x * kCodecWarps + (unsigned long long)warp;
#pragma unroll
    for (int k = 0; k + 1 < kRoundStages; ++k) request(g + (unsigned long long)k * stride, (uint32_t)k);
    uint32_t st = 0, phase = 0;
    EncodeCarry cy;
    cy.pay_used = 0; cy.wide = false;
    while (g < rounds) {
        const At a = at(g);
        const uint32_t nb = (a.len + kBlock - 1) / kBlock;
        if (!mbar_wait(&sh.bar[st], phase)) status |= kStTimeout;
        auto mid = [&]() {
            if (lane == 0) asm volatile("cp.async.bulk.wait_group.read 0;" ::: "memory");
            __syncwarp();
            request(g + (unsigned long long)(kRoundStages - 1) * stride, st == 0 ? (uint32_t)kRoundStages - 1u : st - 1u);
        };
        if (32u * a.rd < nb) {
            uint32_t* slot = ws.slots + (size_t)g * kRoundSlotWords;
            float* stage = sh.stage[st];
            const char* row = reinterpret_cast<const char*>(stage) + 128 * lane;
            const float first = stage[0];
            const float xprev = lane ? read_last_of_row(stage, (uint32_t)lane - 1u) : (a.rd ? sh.front[st][3] : first);
            const uint32_t gslot = (uint32_t)(a.t >> 5);
            cy.pay_used = 0;
            const int rc = encode_round(row, sw, xprev, r, 32u * a.rd + (uint32_t)lane < nb, (uint32_t)lane, 32u, reinterpret_cast<uint32_t*>(stage) - 1,
                                        0u, 1, 9u, (uint32_t)kRoundBufWords - 8u, cy, lane, status, mid);
            if (rc == 0) {
                __syncwarp();
                if (lane == 0) {
                    const uint32_t bytes = (32u + 4u * cy.pay_used + 15u) & ~15u;
                    asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
                    asm volatile("cp.async.bulk.global.shared::cta.bulk_group [%0], [%1], %2;" ::"l"(slot), "r"(smem_u32(stage)), "r"(bytes) : "memory");
                    asm volatile("cp.async.bulk.commit_group;" ::: "memory");
                    ws.round_words[g] = cy.pay_used;
                    atomicAdd(ws.group_acc + gslot, (unsigned long long)cy.pay_used);
                    if (a.rd == 0) ws.outliers[a.t] = (int32_t)(__float_as_uint(__fadd_rn(__fmul_rn(first, r), kRoundMagic)) - kRoundMagicBits);
                }
            } else {
                status |= encode_round_general(x + a.t * sp.T, a.len, a.rd, r, slot, ws.round_words + g, ws.outliers + a.t, ws.group_acc + gslot, lane);
            }
        } else {
            mid();
            if (lane == 0) ws.round_words[g] = 0;   // a round beyond the tile's last block, or no valid bound
        }
        g += stride;
        st = st == (uint32_t)kRoundStages - 1u ? 0u : st + 1u;
        if (st == 0) phase ^= 1u;
    }
    if (lane == 0) asm volatile("cp.async.bulk.wait_group 0;" ::: "memory");
    if (status) atomicOr(ws.status, status);
}

// Step 2: one CTA per group of 32 tiles, a warp per tile, turns the rounds' slots into the group's piece of the
// stream (as place_kernel does for 4096-element tiles; plain loads and stores here, no staging of the payload heads).
__global__ void __launch_bounds__(kPlaceThreads) place_tiled_kernel(uint32_t* __restrict__ out, unsigned long long out_cap, size_t* out_bytes,
                                                                    unsigned long long n, TiledShape sp, uint32_t tiles, Workspace ws, Params hp,
                                                                    int use_dev_params)
{
    __shared__ uint32_t s_words[32], s_part[kPlaceThreads / 32];
    __shared__ unsigned long long s_all[kPlaceThreads / 32];
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    uint32_t status = 0;
    Params prm = hp;
    if (use_dev_params) prm = *ws.params;
    pdl_enter();
    const uint32_t epoch = *reinterpret_cast<volatile uint32_t*>(ws.epoch);
    const uint32_t g = blockIdx.x;
    const uint32_t nT = (uint32_t)((n + sp.T - 1) / sp.T);
    auto put_header = [&](int who, unsigned long long count, uint32_t ntiles) {
        if (who < kHeaderWords) {
            const uint32_t words[kHeaderWords] = {kMagic, kVersion, (uint32_t)count, (uint32_t)(count >> 32), __float_as_uint(prm.eb_abs),
                                                  __float_as_uint(prm.s), sp.T, ntiles};
            uint32_t hv = words[0];
#pragma unroll
            for (int k = 1; k < kHeaderWords; ++k) hv = who == k ? words[k] : hv;
            out[who] = hv;
        }
    };
    auto rearm = [&]() { rearm_groups((tiles >> 5) + 2u, ws, epoch, lane); };   // by one warp, once the CTA has read the group sums it needs
    if (n == 0 || !prm.valid) {   // no elements, or no valid bound: header and length only
        const bool hdr = prm.valid && out_cap >= (unsigned)kHeaderBytes;
        if (tid == 0) *out_bytes = hdr ? kHeaderBytes : 0;
        if (hdr) put_header(tid, 0, 0);
        if (warp == kPlaceThreads / 32 - 1) rearm();
        return;
    }
    const uint32_t t0 = 32u * g;
    const uint32_t ntl = tiles - t0 < 32u ? tiles - t0 : 32u;
    const bool mine = (uint32_t)warp < ntl;
    const uint32_t tile = t0 + (mine ? (uint32_t)warp : 0u);
    const uint32_t len = tiled_len(n, tile, sp.T);
    const uint32_t nb = (len + kBlock - 1) / kBlock, padw = (nb + 3) >> 2;
    const uint32_t* __restrict__ slot0 = ws.slots + (size_t)tile * sp.R * kRoundSlotWords;
    const uint32_t nq = (uint32_t)lane < sp.R ? ws.round_words[(size_t)tile * sp.R + (uint32_t)lane] : 0u;   // lane rd holds round rd's size
    const uint32_t first = (uint32_t)ws.outliers[tile];
    // code-length word w of the tile: blocks 4 w .. 4 w + 3 = word (w & 7) of round w >> 3
    uint32_t lw[2];
#pragma unroll
    for (int k = 0; k < 2; ++k) {
        const uint32_t w = (uint32_t)lane + 32u * k;
        lw[k] = w < padw ? slot0[(size_t)(w >> 3) * kRoundSlotWords + (w & 7u)] : 0u;
    }
    // the payload of the groups in front (this group's place) and of all groups (the stream's size: a stream that does
    // not fit its buffer is not written at all)
    unsigned long long part = 0, all = 0;
    for (uint32_t k = (uint32_t)tid; k < gridDim.x; k += kPlaceThreads) {
        const unsigned long long v = ws.group_acc[k];
        all += v;
        if (k < g) part += v;
    }
#pragma unroll
    for (int d = 16; d >= 1; d >>= 1) { part += __shfl_xor_sync(kFull, part, d); all += __shfl_xor_sync(kFull, all, d); }
    const uint32_t pay = __reduce_add_sync(kFull, nq);
    if (lane == 0) {
        s_words[warp] = mine ? 1u + padw + pay : 0u;
        s_part[warp] = (uint32_t)part;
        s_all[warp] = all;
    }
    __syncthreads();
    if (warp == kPlaceThreads / 32 - 1) rearm();
    const uint32_t wl = s_words[lane];
    const uint32_t incl = warp_incl_scan(wl, lane);
    const uint32_t my_off = __shfl_sync(kFull, incl - wl, warp);
    const uint32_t base = __reduce_add_sync(kFull, s_part[lane]) + g * 32u * (1u + sp.lw_full);   // the tiles in front are full ones
    unsigned long long total = s_all[lane];
#pragma unroll
    for (int d = 16; d >= 1; d >>= 1) total += __shfl_xor_sync(kFull, total, d);
    {
        const uint32_t last_len = tiled_len(n, nT - 1, sp.T);
        const uint32_t last_padw = (((last_len + kBlock - 1) / kBlock) + 3) >> 2;
        total += (unsigned long long)kHeaderWords + nT + (unsigned long long)(nT - 1) * (1u + sp.lw_full) + 1u + last_padw;
    }
    const bool fits = total * 4ull <= out_cap;
    if (!fits && g == 0 && tid == 0) { status |= kStCapacity; *out_bytes = 0; }
    if (mine && fits) {
        const uint32_t words = s_words[warp];
        const unsigned long long word0 = (unsigned long long)kHeaderWords + nT + base + my_off;
        {
            uint32_t* __restrict__ dst = out + word0;
            if (lane == 0) dst[0] = first;
#pragma unroll
            for (int k = 0; k < 2; ++k) {
                const uint32_t w = (uint32_t)lane + 32u * k;
                if (w < padw) dst[1 + w] = lw[k];
            }
            uint32_t* __restrict__ d = dst + 1 + padw;
            for (uint32_t rd = 0; rd < sp.R; ++rd) {
                const uint32_t cnt = __shfl_sync(kFull, nq, (int)rd);
                const uint32_t* __restrict__ src = slot0 + (size_t)rd * kRoundSlotWords + 8;
                // eight loads in flight per lane: a round of mean code length 4 is one trip
                for (uint32_t i0 = 0; i0 < cnt; i0 += 256u) {
                    uint32_t v[8];
#pragma unroll
                    for (int k = 0; k < 8; ++k) {
                        const uint32_t i = i0 + 32u * k + (uint32_t)lane;
                        v[k] = i < cnt ? src[i] : 0u;
                    }
#pragma unroll
                    for (int k = 0; k < 8; ++k) {
                        const uint32_t i = i0 + 32u * k + (uint32_t)lane;
                        if (i < cnt) d[i] = v[k];
                    }
                }
                d += cnt;
            }
            if (lane == 0) out[kHeaderWords + tile] = base + my_off + words;
        }
        if (lane == 0 && tile == nT - 1) *out_bytes = (size_t)((word0 + words) * 4ull);
        if (tile == 0) put_header(lane, n, nT);
    }
    if (status) atomicOr(ws.status, status);
}

// ------------------------------------------------------------------------------------------------ decompress

// describe_blob for tiles of up to 256 blocks (two code-length words per lane): 0 = inconsistent with the blob's size (or
// a code length above 31, or a non-zero padding byte), 1 = consistent and every code of the tile stays below 2^23 in
// magnitude, 2 = consistent, integer arithmetic needed.
__device__ __forceinline__ int describe_blob_wide(const uint32_t* blob, uint32_t words, uint32_t nb, int lane)
{
    const uint32_t padw = (nb + 3) >> 2;
    if (words < 1u + padw) return 0;
    bool bad = false;
    uint32_t sizes = 0, spread = 0;
#pragma unroll
    for (int k = 0; k < 2; ++k) {
        const uint32_t w = (uint32_t)lane + 32u * k;
        const uint32_t lw = w < padw ? blob[1 + w] : 0u;
        bad = bad || (lw & 0xE0E0E0E0u) != 0u;
#pragma unroll
        for (int e = 0; e < 4; ++e) {
            const uint32_t L = (lw >> (8 * e)) & 0xFFu;
            if (4u * w + e >= nb && L) bad = true;
            sizes += L ? L + 1u : 0u;
            spread += L <= 18u ? (32u << L) : (1u << 24);
        }
        spread = min(spread, 1u << 24);
    }
    const uint32_t total = __reduce_add_sync(kFull, sizes);
    spread = __reduce_add_sync(kFull, min(spread, 1u << 24));   // at most 32 * 2^24 = 2^29: no overflow
    if (__any_sync(kFull, bad) || 1u + padw + total != words) return 0;
    const int32_t outlier = (int32_t)blob[0];
    const uint32_t ao = (uint32_t)(outlier < 0 ? -outlier : outlier);
    return (ao < (1u << 23) && spread < (1u << 23)) ? 1 : 2;
}

// A warp decodes a tile of its own, round after round, as decode_tiles_kernel does (blob staged by bulk copies, the
// next tile's into the other of two buffers, a window at a time when it is larger than a buffer; one tensor store per full round of an output on a 16-byte
// boundary, plain coalesced stores otherwise).
__global__ void __launch_bounds__(kCodecThreads, 4) decode_tiles_tiled_kernel(const uint32_t* __restrict__ in, unsigned long long in_cap, TiledShape sp,
                                                                              float* __restrict__ y, unsigned long long y_cap, uint32_t tiles,
                                                                              const __grid_constant__ CUtensorMap map, int mapped, Workspace ws)
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
    // the header, with this launch's tile size in place of the 4096 that read_header insists on
    bool ok = in_cap >= (unsigned long long)kHeaderBytes;
    unsigned long long n = 0;
    uint32_t nT = 0;
    float s = 1.0f;
    if (ok) {
        n = (unsigned long long)ldg_u32(in + 2) | ((unsigned long long)ldg_u32(in + 3) << 32);
        s = __uint_as_float(ldg_u32(in + 5));
        nT = ldg_u32(in + 7);
        ok = ldg_u32(in + 0) == kMagic && ldg_u32(in + 1) == kVersion && ldg_u32(in + 6) == sp.T && (n + sp.T - 1) / sp.T == nT &&
             in_cap >= (unsigned long long)kHeaderBytes + 4ull * nT && s > 0.0f && isfinite(s);
    }
    if (!ok || n > y_cap) {
        if (tid == 0 && blockIdx.x == 0) atomicOr(ws.status, ok ? kStCapacity : kStBadStream);
        return;
    }
    uint32_t fills0 = 0, fills1 = 0;   // bulk copies completed into each blob buffer (phase parities of their mbarriers)
    uint32_t cb = 0;                   // the buffer with the current tile's blob
    const unsigned long long blob0 = (unsigned long long)kHeaderWords + nT;
    const uint32_t last_tile = nT < tiles ? nT : tiles;
    auto request = [&](unsigned long long t, uint32_t buf) {
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
        if (a_end - (uintptr_t)in <= (uintptr_t)in_cap) {
            if (lane == 0) window_request(br, 0, sh.blob[buf], &sh.bar[buf]);
            br.staged = true;
        }
        return br;
    };

    const unsigned long long stride = (unsigned long long)gridDim.x * kCodecWarps;
    unsigned long long t = (unsigned long long)blockIdx.x * kCodecWarps + (unsigned long long)warp;
    BlobRef cur = request(t, 0);
    while (t < last_tile) {
        const unsigned long long tn = t + stride;
        BlobRef nxt;
        nxt.ptr = nullptr; nxt.words = 0; nxt.staged = false;
        if (cur.staged) {
            if (!mbar_wait(&sh.bar[cb], (cb ? fills1 : fills0) & 1u)) status |= kStTimeout;
            if (cb) ++fills1; else ++fills0;
        }
        __syncwarp();
        nxt = request(tn, cb ^ 1u);   // the other blob buffer takes the next tile's blob while this tile is decoded
        if (cur.words == 0xFFFFFFFFu) status |= kStBadStream;
        else if (cur.ptr) {
            const unsigned long long start = t * sp.T;
            const uint32_t len = tiled_len(n, t, sp.T);
            const uint32_t nb = (len + kBlock - 1) / kBlock, padw = (nb + 3) >> 2;
            BlobWindow win;
            win.base = cur.ptr; win.end = cur.words;
            if (cur.staged) win = window_at(cur, 0, sh.blob[cb]);
            const int mode = describe_blob_wide(win.base, cur.words, nb, lane);   // the head (at most 65 words) is in every first window
            if (mode == 0) status |= kStBadStream;
            else {
                uint32_t pay_off = 0;
                int32_t code = (int32_t)win.base[0];
                // the code lengths of the lane's blocks (lane, 32 + lane, ...), one per byte, kept in registers: the window moves away
                uint32_t lp[2] = {0u, 0u};
                {
                    const unsigned char* lb = reinterpret_cast<const unsigned char*>(win.base + 1);
#pragma unroll
                    for (uint32_t e = 0; e < 8u; ++e) {
                        const uint32_t bi = 32u * e + (uint32_t)lane;
                        if (bi < nb) lp[e >> 2] |= (uint32_t)lb[bi] << (8u * (e & 3u));
                    }
                }
                const uint32_t rounds = (nb + 31) >> 5;
                for (uint32_t rd = 0; rd < rounds; ++rd) {
                    const uint32_t L = ((rd < 4u ? lp[0] : lp[1]) >> (8u * (rd & 3u))) & 0xFFu;
                    const uint32_t first = 1u + padw + pay_off;
                    if (win.end < cur.words && first + __reduce_add_sync(kFull, L ? L + 1u : 0u) > win.end) {   // the round reaches past the window
                        __syncwarp();
                        if (lane == 0) window_request(cur, first, sh.blob[cb], &sh.bar[cb]);
                        if (!mbar_wait(&sh.bar[cb], (cb ? fills1 : fills0) & 1u)) status |= kStTimeout;
                        if (cb) ++fills1; else ++fills0;
                        win = window_at(cur, first, sh.blob[cb]);
                    }
                    auto ready = [&]() {   // the one output stage was handed to a tensor store a round ago
                        if (lane == 0) asm volatile("cp.async.bulk.wait_group.read 0;" ::: "memory");
                        __syncwarp();
                    };
                    float* stage = sh.out;
                    if (mode == 1) decode_round<0>(win.base, padw, L, pay_off, code, s, stage, lane, nullptr, ready);
                    else { ready(); decode_round_general(win.base, padw, L, &pay_off, &code, s, stage, lane, nullptr, 0u); }
                    __syncwarp();
                    const uint32_t e0 = rd * (uint32_t)kRound;
                    if (mapped && e0 + (uint32_t)kRound <= len) {
                        if (lane == 0) {
                            asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
                            asm volatile("cp.async.bulk.tensor.2d.global.shared::cta.tile.bulk_group [%0, {%1, %2}], [%3];"
                                         ::"l"(&map), "r"(0), "r"((int)((start + e0) >> 5)), "r"(smem_u32(stage)) : "memory");
                            asm volatile("cp.async.bulk.commit_group;" ::: "memory");
                        }
                    } else {
                        store_round_ragged(y + start + e0, stage, len - e0 < (uint32_t)kRound ? len - e0 : (uint32_t)kRound, lane);
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
