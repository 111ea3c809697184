// C boundary: argument checks, context, job construction and launch order.  Every step of the path itself runs
// in the kernels; nothing here touches data.
#include "../../include/zccl.h"
#include "zccl_internal.h"

#include <cmath>
#include <cstring>
#include <new>
#include <vector>

using namespace zccl;

struct zccl_ctx {
    int device = 0;
    int sm_count = 0;
    size_t max_elems = 0;
    int max_ranks = 0;
    uint32_t debug_epoch = 0;
    uint32_t* gen_sizes = nullptr;        // device: tile sizes (and, behind them, the go flag) of zccl_compress_tiled
    size_t gen_tiles = 0;
    double* quality_partials = nullptr;   // device: per-CTA partial results of zccl_quality
    uint32_t* quality_counter = nullptr;
    Workspace ws{};
    void* small_block = nullptr;     // tile states + counters + params + sizes
    void* slot_block = nullptr;      // round slots, round sizes and outliers of the two-step compression
    uint8_t* arena = nullptr;        // compressed-chunk slots of the emulated ranks
    size_t arena_bytes = 0;
    size_t* sim_sizes = nullptr;     // device: sizes of the last zccl_sim_* call
    int sim_sizes_count = 0;
    int sim_sizes_cap = 0;
    float* stage_x = nullptr;        // device staging of the host-buffer forms
    uint8_t* stage_c = nullptr;
    size_t stage_c_cap = 0;
    size_t* stage_bytes = nullptr;   // device size_t
};

namespace {

inline size_t align_up(size_t v, size_t a) { return (v + a - 1) / a * a; }
inline size_t tiles_of(size_t n) { return (n + kTile - 1) / kTile; }

size_t bound_of(size_t n)
{
    const size_t nT = tiles_of(n);
    size_t total = kHeaderBytes + 4 * nT;
    if (nT == 0) return total;
    const size_t full = nT - 1;
    total += full * (4 + kBlocksPerTile + (size_t)kBlocksPerTile * 128);
    const size_t len = n - full * kTile;
    const size_t nb = (len + kBlock - 1) / kBlock;
    total += 4 + ((nb + 3) & ~(size_t)3) + nb * 128;
    return total;
}

// eb -> (eb_abs, s, r) for an absolute bound, with the same IEEE operations the device uses for relative bounds.
int resolve_abs_host(float eb, Params& p)
{
    volatile float ebq = eb * 0.984375f;
    volatile float s = ebq * 2.0f;
    if (!(s > 0.0f) || !std::isfinite((float)s)) return ZCCL_E_DEGENERATE;
    volatile float r = 1.0f / s;
    if (!std::isfinite((float)r)) return ZCCL_E_DEGENERATE;
    p.eb_abs = eb; p.s = s; p.r = r; p.valid = 1;
    return ZCCL_OK;
}

inline bool eb_ok(int mode, float eb)
{
    if (mode == ZCCL_EB_RESOLVED) return true;   // the bound is the context's resolved block; eb is not looked at
    return (mode == ZCCL_EB_ABS || mode == ZCCL_EB_REL) && eb > 0.0f && std::isfinite(eb);
}

inline int cuda_rc(cudaError_t e) { return e == cudaSuccess ? ZCCL_OK : ZCCL_E_CUDA; }

// Collects jobs and launches them in batches of at most kMaxJobs.
template <int CAP>
struct BatcherT {
    JobBatchT<CAP> jb{};
    void reset() { jb.count = 0; jb.total_tiles = 0; }
    BatcherT() { reset(); }
    bool full() const { return jb.count == CAP; }
    void add(const Job& j, size_t tiles)
    {
        Job& d = jb.job[jb.count++];
        d = j;
        d.tile_begin = jb.total_tiles;
        jb.total_tiles += (uint32_t)(tiles ? tiles : 1);
    }
};

using Batcher = BatcherT<kMaxJobs>;
using DecodeBatcher = BatcherT<kMaxDecodeJobs>;

struct RangeList {
    std::vector<const float*> x;
    std::vector<size_t> n;
};

// Resolves the bound: ABS on the host, REL by a device min/max pass over all listed buffers.
int resolve_bound(zccl_ctx* c, const RangeList& rl, int mode, float eb, Params& hp, bool& on_device, cudaStream_t st)
{
    on_device = false;
    if (mode == ZCCL_EB_ABS) return resolve_abs_host(eb, hp);
    if (mode == ZCCL_EB_RESOLVED) {     // zccl_resolve_range (or an earlier ZCCL_EB_REL call) left the bound on the device
        hp = Params{0.f, 1.f, 1.f, 1};
        on_device = true;
        return ZCCL_OK;
    }
    size_t total = 0;
    for (size_t v : rl.n) total += v;
    if (total == 0) return ZCCL_E_DEGENERATE;
    RangeBatch rb{};
    rb.count = 0;
    for (size_t i = 0; i < rl.x.size(); ++i) {
        if (rl.n[i] == 0) continue;
        if (rb.count == kMaxJobs) {     // a full batch with more to come: collect only
            rb.finish = kRangeOnly;
            if (launch_range(rb, c->ws, c->sm_count, st) != cudaSuccess) return ZCCL_E_CUDA;
            rb.count = 0;
        }
        rb.x[rb.count] = rl.x[i];
        rb.n[rb.count] = rl.n[i];
        ++rb.count;
    }
    rb.finish = kRangeResolve;          // the last launch also turns (min, max, eb) into the bound
    rb.eb = eb;
    if (launch_range(rb, c->ws, c->sm_count, st) != cudaSuccess) return ZCCL_E_CUDA;
    hp = Params{0.f, 1.f, 1.f, 1};
    on_device = true;
    return ZCCL_OK;
}

int flush_encode(zccl_ctx* c, Batcher& b, EncodeMode mode, bool dev_params, const Params& hp, cudaStream_t st)
{
    if (b.jb.count == 0) return ZCCL_OK;
    if (b.jb.total_tiles > c->ws.max_tiles) return ZCCL_E_ARG;
    cudaError_t e = launch_encode(b.jb, mode, c->ws, dev_params, hp, c->sm_count, st);
    b.reset();
    return cuda_rc(e);
}
int flush_decode(zccl_ctx* c, Batcher& b, cudaStream_t st)
{
    if (b.jb.count == 0) return ZCCL_OK;
    cudaError_t e = launch_decode(b.jb, c->ws, c->sm_count, st);
    b.reset();
    return cuda_rc(e);
}
int flush_decode(zccl_ctx* c, DecodeBatcher& b, cudaStream_t st)
{
    if (b.jb.count == 0) return ZCCL_OK;
    cudaError_t e = launch_decode_wide(b.jb, c->ws, c->sm_count, st);
    b.reset();
    return cuda_rc(e);
}
struct CopyBatcher {
    CopyBatch cb{};
    CopyBatcher() { cb.count = 0; }
    void add(const void* src, void* dst, const size_t* bytes, size_t* bytes_out, size_t cap)
    {
        CopyJob& j = cb.job[cb.count++];
        j.src = (const uint32_t*)src; j.dst = (uint32_t*)dst; j.bytes = bytes; j.bytes_out = bytes_out; j.cap = cap;
        j.fixed_bytes = 0;
    }
    void add_fixed(const void* src, void* dst, size_t nbytes)   // a copy whose length the host knows
    {
        CopyJob& j = cb.job[cb.count++];
        j.src = (const uint32_t*)src; j.dst = (uint32_t*)dst; j.bytes = nullptr; j.bytes_out = nullptr; j.cap = nbytes;
        j.fixed_bytes = nbytes;
    }
    bool full() const { return cb.count == kMaxJobs; }
};
int flush_copy(zccl_ctx* c, CopyBatcher& b, cudaStream_t st)
{
    if (b.cb.count == 0) return ZCCL_OK;
    cudaError_t e = launch_copy(b.cb, c->ws, c->sm_count, st);
    b.cb.count = 0;
    return cuda_rc(e);
}

inline void chunk_span(size_t n, int N, int c, size_t& off, size_t& len)
{
    const size_t m = (n + (size_t)N - 1) / (size_t)N;
    size_t o = (size_t)c * m;
    if (o > n) o = n;
    off = o;
    len = (n - o < m) ? n - o : m;
}

}  // namespace

extern "C" {

size_t zccl_compress_bound(size_t n) { return bound_of(n); }

unsigned long long zccl_launch_count(void) { return launch_count(); }

const char* zccl_strerror(int code)
{
    switch (code) {
        case ZCCL_OK: return "ok";
        case ZCCL_E_ARG: return "invalid argument";
        case ZCCL_E_CUDA: return "CUDA runtime error";
        case ZCCL_E_CAPACITY: return "output capacity too small";
        case ZCCL_E_RANGE: return "value out of quantisable range";
        case ZCCL_E_BAD_STREAM: return "malformed compressed stream";
        case ZCCL_E_TIMEOUT: return "placement scan timed out";
        case ZCCL_E_DEGENERATE: return "degenerate value range or step";
        case ZCCL_E_TOO_LARGE: return "more elements than the allocation-free entry point supports";
        case ZCCL_W_PRECISION: return "warning: codes beyond 2^15, bound may be exceeded by fp32 rounding";
        default: return "unknown status";
    }
}

int zccl_ctx_create(zccl_ctx** out, size_t max_elems, int max_ranks)
{
    if (!out || max_elems == 0 || max_ranks < 0 || max_ranks > ZCCL_MAX_RANKS) return ZCCL_E_ARG;
    zccl_ctx* c = new (std::nothrow) zccl_ctx();
    if (!c) return ZCCL_E_ARG;
    if (cudaGetDevice(&c->device) != cudaSuccess) { delete c; return ZCCL_E_CUDA; }
    cudaDeviceProp prop;
    if (cudaGetDeviceProperties(&prop, c->device) != cudaSuccess) { delete c; return ZCCL_E_CUDA; }
    c->sm_count = prop.multiProcessorCount;
    c->max_elems = max_elems;
    c->max_ranks = max_ranks;

    const size_t max_tiles = tiles_of(max_elems) + (size_t)(max_ranks > kMaxJobs ? max_ranks : kMaxJobs) + 64;
    if (max_tiles > 0xFFFFFFFFull) { delete c; return ZCCL_E_ARG; }
    c->sim_sizes_cap = 2 * (max_ranks > 1 ? max_ranks * max_ranks : 1) + 2;
    const size_t off_state = 0;
    const size_t off_group = off_state + 8 * max_tiles;
    const size_t off_acc = off_group + 8 * (size_t)group_slots(max_tiles);
    const size_t off_small = align_up(off_acc + 8 * (size_t)group_slots(4 * max_tiles), 256);   // groups of 32 tiles of 1024 elements at most
    const size_t off_sizes = off_small + 256;
    const size_t off_quality = align_up(off_sizes + sizeof(size_t) * (size_t)(c->sim_sizes_cap + 1), 256);
    const size_t small_bytes = off_quality + sizeof(double) * 4 * (size_t)kQualityCtas + 256;
    bool ok = cudaMalloc(&c->small_block, small_bytes) == cudaSuccess;
    if (ok) ok = cudaMemset(c->small_block, 0, small_bytes) == cudaSuccess;
    if (ok) {
        uint8_t* b = (uint8_t*)c->small_block;
        c->ws.tile_state = (unsigned long long*)(b + off_state);
        c->ws.group_state = (unsigned long long*)(b + off_group);
        c->ws.group_acc = (unsigned long long*)(b + off_acc);
        uint32_t* sm = (uint32_t*)(b + off_small);
        c->ws.ticket = sm + 0;
        c->ws.done = sm + 1;
        c->ws.epoch = sm + 2;
        c->ws.status = sm + 3;
        c->ws.params = (Params*)(sm + 4);
        c->ws.minmax = sm + 8;
        c->ws.params64 = (ParamsF64*)(b + off_small + 64);
        c->ws.minmax64 = (unsigned long long*)(b + off_small + 96);
        c->ws.max_tiles = (uint32_t)max_tiles;
        c->ws.skip_publish = 0xFFFFFFFFu;
        c->sim_sizes = (size_t*)(b + off_sizes);
        c->stage_bytes = c->sim_sizes + c->sim_sizes_cap;
        c->quality_partials = (double*)(b + off_quality);
        c->quality_counter = (uint32_t*)(b + off_quality + sizeof(double) * 4 * (size_t)kQualityCtas);
        const uint32_t init[3] = {1u, 0xFFFFFFFFu, 0u};   // epoch, min key, max key
        const unsigned long long init64[2] = {0xFFFFFFFFFFFFFFFFull, 0ull};
        ok = cudaMemcpy(c->ws.epoch, &init[0], 4, cudaMemcpyHostToDevice) == cudaSuccess &&
             cudaMemcpy(c->ws.minmax, &init[1], 8, cudaMemcpyHostToDevice) == cudaSuccess &&
             cudaMemcpy(c->ws.minmax64, init64, 16, cudaMemcpyHostToDevice) == cudaSuccess;
    }
    if (ok) {
        const size_t off_rw = align_up(max_tiles * 4 * (size_t)kRoundSlotWords * 4, 256);
        const size_t off_ol = align_up(off_rw + max_tiles * 4 * 4, 256);
        ok = cudaMalloc(&c->slot_block, off_ol + max_tiles * 4 * 4) == cudaSuccess;   // a first code per tile, tiles of 1024 elements at most
        if (ok) {
            uint8_t* b = (uint8_t*)c->slot_block;
            c->ws.slots = (uint32_t*)b;
            c->ws.round_words = (uint32_t*)(b + off_rw);
            c->ws.outliers = (int32_t*)(b + off_ol);
        }
    }
    if (ok && max_ranks >= 2) {
        c->arena_bytes = (size_t)(max_ranks + 2) * align_up(bound_of(max_elems) + (size_t)max_ranks * 1024, 256);
        ok = cudaMalloc((void**)&c->arena, c->arena_bytes) == cudaSuccess;
    }
    if (ok) {
        c->gen_tiles = (max_elems + kGenericMinTile - 1) / kGenericMinTile + 1;
        ok = cudaMalloc((void**)&c->gen_sizes, sizeof(uint32_t) * (c->gen_tiles + 1)) == cudaSuccess;
    }
    if (ok) {
        c->stage_c_cap = align_up(bound_of(max_elems), 256);
        ok = cudaMalloc((void**)&c->stage_x, sizeof(float) * max_elems) == cudaSuccess &&
             cudaMalloc((void**)&c->stage_c, c->stage_c_cap) == cudaSuccess;
    }
    if (!ok) { zccl_ctx_destroy(c); return ZCCL_E_CUDA; }
    *out = c;
    return ZCCL_OK;
}

void zccl_ctx_destroy(zccl_ctx* c)
{
    if (!c) return;
    cudaDeviceSynchronize();
    if (c->small_block) cudaFree(c->small_block);
    if (c->slot_block) cudaFree(c->slot_block);
    if (c->gen_sizes) cudaFree(c->gen_sizes);
    if (c->arena) cudaFree(c->arena);
    if (c->stage_x) cudaFree(c->stage_x);
    if (c->stage_c) cudaFree(c->stage_c);
    delete c;
}

int zccl_status(zccl_ctx* c, void* stream)
{
    if (!c) return ZCCL_E_ARG;
    cudaStream_t st = (cudaStream_t)stream;
    uint32_t bits = 0;
    if (cudaMemcpyAsync(&bits, c->ws.status, 4, cudaMemcpyDeviceToHost, st) != cudaSuccess) return ZCCL_E_CUDA;
    if (cudaMemsetAsync(c->ws.status, 0, 4, st) != cudaSuccess) return ZCCL_E_CUDA;
    if (cudaStreamSynchronize(st) != cudaSuccess) return ZCCL_E_CUDA;
    if (bits & kStTimeout) return ZCCL_E_TIMEOUT;
    if (bits & kStDegenerate) return ZCCL_E_DEGENERATE;   // the cause of the empty streams that later calls then reject
    if (bits & kStBadStream) return ZCCL_E_BAD_STREAM;
    if (bits & kStRange) return ZCCL_E_RANGE;
    if (bits & kStCapacity) return ZCCL_E_CAPACITY;
    if (bits & kStPrecision) return ZCCL_W_PRECISION;
    return ZCCL_OK;
}

int zccl_debug_skip_publish(zccl_ctx* c, long long tile)
{
    if (!c) return ZCCL_E_ARG;
    c->ws.skip_publish = (tile < 0 || tile >= 0xFFFFFFFFll) ? 0xFFFFFFFFu : (uint32_t)tile;
    return ZCCL_OK;
}

int zccl_debug_set_launch_counter(zccl_ctx* c, unsigned int value, void* stream)
{
    if (!c || value == 0 || value > 0x7FFFFFFFu) return ZCCL_E_ARG;
    c->debug_epoch = value;   // the source of an asynchronous copy must outlive the call
    return cuda_rc(cudaMemcpyAsync(c->ws.epoch, &c->debug_epoch, sizeof(uint32_t), cudaMemcpyHostToDevice, (cudaStream_t)stream));
}

int zccl_compress(zccl_ctx* c, const float* x, size_t n, int eb_mode, float eb,
                  void* out, size_t out_capacity, size_t* out_bytes, void* stream)
{
    if (!c || !out || !out_bytes || (!x && n) || !eb_ok(eb_mode, eb) || n > c->max_elems) return ZCCL_E_ARG;
    if (((uintptr_t)out & 3u) || ((uintptr_t)x & 3u)) return ZCCL_E_ARG;
    if (out_capacity < kHeaderBytes + 4 * tiles_of(n)) return ZCCL_E_CAPACITY;
    cudaStream_t st = (cudaStream_t)stream;
    Params hp{};
    bool dev = false;
    RangeList rl;
    rl.x.push_back(x); rl.n.push_back(n);
    int rc = resolve_bound(c, rl, eb_mode, eb, hp, dev, st);
    if (rc != ZCCL_OK) return rc;
    Batcher b;
    Job j{};
    j.x = x; j.out = (uint32_t*)out; j.out_bytes = out_bytes; j.n = n; j.out_cap = out_capacity;
    b.add(j, tiles_of(n));
    return flush_encode(c, b, kEncodeRaw, dev, hp, st);
}

int zccl_decompress(zccl_ctx* c, const void* in, size_t in_bytes_max, float* y, size_t y_capacity_elems, void* stream)
{
    if (!c || !in || (!y && y_capacity_elems)) return ZCCL_E_ARG;
    if (((uintptr_t)in & 3u) || ((uintptr_t)y & 3u)) return ZCCL_E_ARG;
    if (in_bytes_max < (size_t)kHeaderBytes) return ZCCL_E_CAPACITY;
    if (tiles_of(y_capacity_elems) >= 0xFFFFFFFFull) return ZCCL_E_ARG;
    Batcher b;
    Job j{};
    j.in_c = (const uint32_t*)in; j.in_cap = in_bytes_max; j.y = y; j.n = y_capacity_elems;
    b.add(j, tiles_of(y_capacity_elems));
    return flush_decode(c, b, (cudaStream_t)stream);
}

int zccl_decompress_reduce_compress(zccl_ctx* c, const void* in_c, size_t in_bytes_max,
                                    const float* local, const void* local_c, size_t local_c_bytes_max, size_t n,
                                    void* out_c, size_t out_capacity, size_t* out_bytes,
                                    float* raw_out, unsigned flags, void* stream)
{
    if (!c || !in_c || !out_c || !out_bytes || n > c->max_elems) return ZCCL_E_ARG;
    if ((local == nullptr) == (local_c == nullptr)) return ZCCL_E_ARG;
    if (((uintptr_t)in_c & 3u) || ((uintptr_t)local & 3u) || ((uintptr_t)local_c & 3u) || ((uintptr_t)out_c & 3u) ||
        ((uintptr_t)raw_out & 3u)) return ZCCL_E_ARG;
    if (in_bytes_max < (size_t)kHeaderBytes || (local_c && local_c_bytes_max < (size_t)kHeaderBytes)) return ZCCL_E_CAPACITY;
    if (out_capacity < kHeaderBytes + 4 * tiles_of(n)) return ZCCL_E_CAPACITY;
    Batcher b;
    Job j{};
    j.x = local; j.in_c = (const uint32_t*)in_c; j.in_c2 = (const uint32_t*)local_c;
    j.in_cap = in_bytes_max; j.in2_cap = local_c_bytes_max;
    j.out = (uint32_t*)out_c; j.out_cap = out_capacity; j.out_bytes = out_bytes; j.y = raw_out; j.n = n; j.flags = flags;
    b.add(j, tiles_of(n));
    return flush_encode(c, b, kEncodeFused, false, Params{0.f, 1.f, 1.f, 1}, (cudaStream_t)stream);
}

int zccl_sim_allreduce(zccl_ctx* c, const float* const* send, float* const* recv, int N,
                       size_t n, int eb_mode, float eb, unsigned flags, void* stream)
{
    if (!c || !send || !recv || N < 1 || N > c->max_ranks || !eb_ok(eb_mode, eb) || n > c->max_elems) return ZCCL_E_ARG;
    for (int r = 0; r < N; ++r) if (!send[r] || !recv[r]) return ZCCL_E_ARG;
    cudaStream_t st = (cudaStream_t)stream;
    const size_t m = (n + (size_t)N - 1) / (size_t)N;
    const size_t slot = align_up(bound_of(m), 256);
    const size_t need = ((size_t)N * N + 2 * (size_t)N) * slot;
    if (need > c->arena_bytes) return ZCCL_E_ARG;
    uint8_t* cur0 = c->arena;
    uint8_t* nxt0 = c->arena + (size_t)N * slot;
    uint8_t* gs0 = c->arena + 2 * (size_t)N * slot;
    auto gslot = [&](int r, int ch) { return gs0 + ((size_t)r * N + ch) * slot; };
    size_t* hop_sz = c->sim_sizes;                       // [N][N]: step k, rank r
    size_t* g_sz = c->sim_sizes + (size_t)N * N;         // [N][N]: rank r, chunk ch
    c->sim_sizes_count = N * N;
    if (cudaMemsetAsync(c->sim_sizes, 0, sizeof(size_t) * 2 * (size_t)N * N, st) != cudaSuccess) return ZCCL_E_CUDA;

    Params hp{};
    bool dev = false;
    RangeList rl;
    for (int r = 0; r < N; ++r) { rl.x.push_back(send[r]); rl.n.push_back(n); }
    int rc = resolve_bound(c, rl, eb_mode, eb, hp, dev, st);
    if (rc != ZCCL_OK) return rc;

    // step 0: rank r compresses its chunk r
    Batcher b;
    for (int r = 0; r < N; ++r) {
        size_t off, len; chunk_span(n, N, r, off, len);
        Job j{};
        j.x = send[r] + off; j.n = len; j.out = (uint32_t*)(cur0 + (size_t)r * slot); j.out_cap = slot;
        j.out_bytes = hop_sz + r;
        b.add(j, tiles_of(len));
        if (b.full() && (rc = flush_encode(c, b, kEncodeRaw, dev, hp, st)) != ZCCL_OK) return rc;
    }
    if ((rc = flush_encode(c, b, kEncodeRaw, dev, hp, st)) != ZCCL_OK) return rc;
    if (N == 1) return cuda_rc(cudaMemcpyAsync(recv[0], send[0], sizeof(float) * n, cudaMemcpyDeviceToDevice, st));

    // reduce-scatter hops: fused decode + add own chunk + re-encode
    uint8_t* cur = cur0;
    uint8_t* nxt = nxt0;
    for (int k = 0; k + 1 < N; ++k) {
        const bool last = (k == N - 2);
        for (int r = 0; r < N; ++r) {
            const int from = (r - 1 + N) % N;
            const int ch = ((r - k - 1) % N + N) % N;
            size_t off, len; chunk_span(n, N, ch, off, len);
            Job j{};
            j.in_c = (const uint32_t*)(cur + (size_t)from * slot); j.in_cap = slot;
            j.x = send[r] + off; j.n = len;
            j.out = (uint32_t*)(nxt + (size_t)r * slot); j.out_cap = slot;
            j.out_bytes = hop_sz + (size_t)(k + 1) * N + r;
            j.y = last ? recv[r] + off : nullptr;
            j.flags = flags;
            b.add(j, tiles_of(len));
            if (b.full() && (rc = flush_encode(c, b, kEncodeFused, false, hp, st)) != ZCCL_OK) return rc;
        }
        if ((rc = flush_encode(c, b, kEncodeFused, false, hp, st)) != ZCCL_OK) return rc;
        uint8_t* t = cur; cur = nxt; nxt = t;
    }

    // allgather stage: N-1 forwarding hops of compressed chunks between per-rank slots, all in one launch.  Rank r
    // owns chunk (r+1) mod N in cur[r]; hop h hands it to rank r+1+h.
    const size_t* own_sz = hop_sz + (size_t)(N - 1) * N;
    {
        ChainBatch cb{};
        cb.slots = gs0; cb.sizes = g_sz; cb.slot_bytes = slot; cb.N = N; cb.hops = N - 1; cb.count = N;
        for (int r = 0; r < N; ++r) {
            ChainJob& j = cb.job[r];
            j.src0 = (const uint32_t*)(cur + (size_t)r * slot); j.bytes = own_sz + r; j.first_rank = (r + 1) % N; j.chunk = (r + 1) % N;
        }
        if ((rc = cuda_rc(launch_copy_chain(cb, c->ws, c->sm_count, st))) != ZCCL_OK) return rc;
    }
    // every rank decompresses the chunks it does not own
    DecodeBatcher db;
    for (int r = 0; r < N; ++r) {
        for (int ch = 0; ch < N; ++ch) {
            if (ch == (r + 1) % N) continue;
            size_t off, len; chunk_span(n, N, ch, off, len);
            Job j{};
            j.in_c = (const uint32_t*)gslot(r, ch); j.in_cap = slot; j.y = recv[r] + off; j.n = len;
            db.add(j, tiles_of(len));
            if (db.full() && (rc = flush_decode(c, db, st)) != ZCCL_OK) return rc;
        }
    }
    if ((rc = flush_decode(c, db, st)) != ZCCL_OK) return rc;
    if ((flags & ZCCL_OP_MASK) == ZCCL_OP_AVG) {   // Average = Sum / N: one division per element of every rank's result
        ScaleBatch sb{};
        sb.n = n; sb.divisor = (float)N; sb.count = 0;
        for (int r = 0; r < N; ++r) {
            sb.y[sb.count++] = recv[r];
            if (sb.count == kMaxJobs) {
                if (launch_scale(sb, c->sm_count, st) != cudaSuccess) return ZCCL_E_CUDA;
                sb.count = 0;
            }
        }
        if (launch_scale(sb, c->sm_count, st) != cudaSuccess) return ZCCL_E_CUDA;
    }
    return ZCCL_OK;
}

int zccl_sim_allgather(zccl_ctx* c, const float* const* send, float* const* recv, int N,
                       size_t n, int eb_mode, float eb, void* stream)
{
    if (!c || !send || !recv || N < 1 || N > c->max_ranks || !eb_ok(eb_mode, eb) || n * (size_t)N > c->max_elems)
        return ZCCL_E_ARG;
    for (int r = 0; r < N; ++r) if (!send[r] || !recv[r]) return ZCCL_E_ARG;
    cudaStream_t st = (cudaStream_t)stream;
    const size_t slot = align_up(bound_of(n), 256);
    if ((size_t)N * N * slot > c->arena_bytes) return ZCCL_E_ARG;
    auto gslot = [&](int r, int src) { return c->arena + ((size_t)r * N + src) * slot; };
    size_t* own_sz = c->sim_sizes;                     // [N]
    size_t* g_sz = c->sim_sizes + N;                   // [N][N]
    c->sim_sizes_count = N;
    if (cudaMemsetAsync(c->sim_sizes, 0, sizeof(size_t) * ((size_t)N * N + N), st) != cudaSuccess) return ZCCL_E_CUDA;

    Params hp{};
    bool dev = false;
    RangeList rl;
    for (int r = 0; r < N; ++r) { rl.x.push_back(send[r]); rl.n.push_back(n); }
    int rc = resolve_bound(c, rl, eb_mode, eb, hp, dev, st);
    if (rc != ZCCL_OK) return rc;

    Batcher b;
    for (int r = 0; r < N; ++r) {   // compress once
        Job j{};
        j.x = send[r]; j.n = n; j.out = (uint32_t*)gslot(r, r); j.out_cap = slot; j.out_bytes = own_sz + r;
        b.add(j, tiles_of(n));
        if (b.full() && (rc = flush_encode(c, b, kEncodeRaw, dev, hp, st)) != ZCCL_OK) return rc;
    }
    if ((rc = flush_encode(c, b, kEncodeRaw, dev, hp, st)) != ZCCL_OK) return rc;

    if (N > 1) {   // forward compressed bytes around the ring: hop h hands rank r's contribution to rank r+1+h
        ChainBatch cb{};
        cb.slots = c->arena; cb.sizes = g_sz; cb.slot_bytes = slot; cb.N = N; cb.hops = N - 1; cb.count = N;
        for (int r = 0; r < N; ++r) {
            ChainJob& j = cb.job[r];
            j.src0 = (const uint32_t*)gslot(r, r); j.bytes = own_sz + r; j.first_rank = (r + 1) % N; j.chunk = r;
        }
        // own contributions stay uncompressed: their copies ride along in the forwarding launch when they fit its grid
        CopyBatcher own;
        if (N <= kMaxJobs)
            for (int r = 0; r < N; ++r) own.add_fixed(send[r], recv[r] + (size_t)r * n, sizeof(float) * n);
        if ((rc = cuda_rc(launch_copy_chain(cb, c->ws, c->sm_count, st, N <= kMaxJobs ? &own.cb : nullptr))) != ZCCL_OK) return rc;
    }
    if (N == 1 || N > kMaxJobs) {   // ... or take a launch of their own
        CopyBatcher cb;
        for (int r = 0; r < N; ++r) {
            cb.add_fixed(send[r], recv[r] + (size_t)r * n, sizeof(float) * n);
            if (cb.full() && (rc = flush_copy(c, cb, st)) != ZCCL_OK) return rc;
        }
        if ((rc = flush_copy(c, cb, st)) != ZCCL_OK) return rc;
    }
    DecodeBatcher db;
    for (int r = 0; r < N; ++r) {
        for (int src = 0; src < N; ++src) {
            if (src == r) continue;
            Job j{};
            j.in_c = (const uint32_t*)gslot(r, src); j.in_cap = slot; j.y = recv[r] + (size_t)src * n; j.n = n;
            db.add(j, tiles_of(n));
            if (db.full() && (rc = flush_decode(c, db, st)) != ZCCL_OK) return rc;
        }
    }
    return flush_decode(c, db, st);
}

int zccl_sim_bcast(zccl_ctx* c, const float* root, float* const* recv, int nsinks, size_t n,
                   int eb_mode, float eb, void* stream)
{
    if (!c || (!root && n) || !recv || nsinks < 0 || nsinks > c->max_ranks || !eb_ok(eb_mode, eb) || n > c->max_elems)
        return ZCCL_E_ARG;
    for (int r = 0; r < nsinks; ++r) if (!recv[r]) return ZCCL_E_ARG;
    cudaStream_t st = (cudaStream_t)stream;
    const size_t slot = align_up(bound_of(n), 256);
    if ((size_t)(nsinks + 1) * slot > c->arena_bytes) return ZCCL_E_ARG;
    auto rslot = [&](int rank) { return c->arena + (size_t)rank * slot; };   // rank 0 = root, sinks are 1..nsinks
    size_t* sz = c->sim_sizes;   // [nsinks + 1]
    c->sim_sizes_count = 1;
    if (cudaMemsetAsync(c->sim_sizes, 0, sizeof(size_t) * (size_t)(nsinks + 1), st) != cudaSuccess) return ZCCL_E_CUDA;
    int rc = zccl_compress(c, root, n, eb_mode, eb, rslot(0), slot, sz, stream);
    if (rc != ZCCL_OK) return rc;
    CopyBatcher cb;
    for (int dist = 1; dist <= nsinks; dist <<= 1) {   // binomial tree: holders forward to rank + dist
        for (int src = 0; src < dist; ++src) {
            const int dst = src + dist;
            if (dst > nsinks) break;
            cb.add(rslot(src), rslot(dst), sz + src, sz + dst, slot);
            if (cb.full() && (rc = flush_copy(c, cb, st)) != ZCCL_OK) return rc;
        }
        if ((rc = flush_copy(c, cb, st)) != ZCCL_OK) return rc;
    }
    Batcher b;
    for (int k = 0; k < nsinks; ++k) {
        Job j{};
        j.in_c = (const uint32_t*)rslot(k + 1); j.in_cap = slot; j.y = recv[k]; j.n = n;
        b.add(j, tiles_of(n));
        if (b.full() && (rc = flush_decode(c, b, st)) != ZCCL_OK) return rc;
    }
    return flush_decode(c, b, st);
}

int zccl_sim_reduce_scatter(zccl_ctx* c, const float* const* send, float* const* recv, int N,
                            size_t n, int eb_mode, float eb, void* stream)
{
    if (!c || !send || !recv || N < 1 || N > c->max_ranks || !eb_ok(eb_mode, eb) || n > c->max_elems) return ZCCL_E_ARG;
    for (int r = 0; r < N; ++r) if (!send[r] || !recv[r]) return ZCCL_E_ARG;
    cudaStream_t st = (cudaStream_t)stream;
    const size_t m = (n + (size_t)N - 1) / (size_t)N;
    const size_t slot = align_up(bound_of(m), 256);
    if (2 * (size_t)N * slot > c->arena_bytes) return ZCCL_E_ARG;
    uint8_t* cur = c->arena;
    uint8_t* nxt = c->arena + (size_t)N * slot;
    size_t* hop_sz = c->sim_sizes;                       // [N-1][N]: step k, rank r; one more row for the last hop's unused stream
    c->sim_sizes_count = (N - 1) * N;
    if (cudaMemsetAsync(c->sim_sizes, 0, sizeof(size_t) * (size_t)N * N, st) != cudaSuccess) return ZCCL_E_CUDA;
    if (N == 1) {
        size_t off, len; chunk_span(n, N, 0, off, len);
        return cuda_rc(cudaMemcpyAsync(recv[0], send[0], sizeof(float) * len, cudaMemcpyDeviceToDevice, st));
    }

    Params hp{};
    bool dev = false;
    RangeList rl;
    for (int r = 0; r < N; ++r) { rl.x.push_back(send[r]); rl.n.push_back(n); }
    int rc = resolve_bound(c, rl, eb_mode, eb, hp, dev, st);
    if (rc != ZCCL_OK) return rc;

    Batcher b;
    for (int r = 0; r < N; ++r) {   // step 0: rank r compresses chunk r-1
        size_t off, len; chunk_span(n, N, (r - 1 + N) % N, off, len);
        Job j{};
        j.x = send[r] + off; j.n = len; j.out = (uint32_t*)(cur + (size_t)r * slot); j.out_cap = slot;
        j.out_bytes = hop_sz + r;
        b.add(j, tiles_of(len));
        if (b.full() && (rc = flush_encode(c, b, kEncodeRaw, dev, hp, st)) != ZCCL_OK) return rc;
    }
    if ((rc = flush_encode(c, b, kEncodeRaw, dev, hp, st)) != ZCCL_OK) return rc;
    for (int k = 0; k + 1 < N; ++k) {   // step k+1: rank r takes chunk r-k-2 from rank r-1; the last step keeps the sum
        const bool last = (k == N - 2);
        for (int r = 0; r < N; ++r) {
            const int from = (r - 1 + N) % N;
            const int ch = ((r - k - 2) % N + N) % N;
            size_t off, len; chunk_span(n, N, ch, off, len);
            Job j{};
            j.in_c = (const uint32_t*)(cur + (size_t)from * slot); j.in_cap = slot;
            j.x = send[r] + off; j.n = len;
            j.out = (uint32_t*)(nxt + (size_t)r * slot); j.out_cap = slot;
            j.out_bytes = hop_sz + (size_t)(k + 1) * N + r;   // the last step's stream is produced but not part of the collective
            j.y = last ? recv[r] : nullptr;
            j.flags = 0;
            b.add(j, tiles_of(len));
            if (b.full() && (rc = flush_encode(c, b, kEncodeFused, false, hp, st)) != ZCCL_OK) return rc;
        }
        if ((rc = flush_encode(c, b, kEncodeFused, false, hp, st)) != ZCCL_OK) return rc;
        uint8_t* t = cur; cur = nxt; nxt = t;
    }
    return ZCCL_OK;
}

int zccl_sim_scatter(zccl_ctx* c, const float* root, float* const* recv, int N, size_t n,
                     int eb_mode, float eb, void* stream)
{
    if (!c || (!root && n) || !recv || N < 1 || N > c->max_ranks || !eb_ok(eb_mode, eb) || n * (size_t)N > c->max_elems)
        return ZCCL_E_ARG;
    for (int r = 0; r < N; ++r) if (!recv[r]) return ZCCL_E_ARG;
    cudaStream_t st = (cudaStream_t)stream;
    const size_t slot = align_up(bound_of(n), 256);
    if ((size_t)N * N * slot > c->arena_bytes) return ZCCL_E_ARG;
    auto gslot = [&](int r, int ch) { return c->arena + ((size_t)r * N + ch) * slot; };
    size_t* own_sz = c->sim_sizes;                     // [N]: bytes of chunk c as compressed by the root
    size_t* g_sz = c->sim_sizes + N;                   // [N][N]: rank r, chunk c
    c->sim_sizes_count = N;
    if (cudaMemsetAsync(c->sim_sizes, 0, sizeof(size_t) * ((size_t)N * N + N), st) != cudaSuccess) return ZCCL_E_CUDA;

    Params hp{};
    bool dev = false;
    RangeList rl;
    rl.x.push_back(root); rl.n.push_back(n * (size_t)N);
    int rc = resolve_bound(c, rl, eb_mode, eb, hp, dev, st);
    if (rc != ZCCL_OK) return rc;

    Batcher b;
    for (int ch = 1; ch < N; ++ch) {   // the root compresses every foreign chunk once
        Job j{};
        j.x = root + (size_t)ch * n; j.n = n; j.out = (uint32_t*)gslot(0, ch); j.out_cap = slot; j.out_bytes = own_sz + ch;
        b.add(j, tiles_of(n));
        if (b.full() && (rc = flush_encode(c, b, kEncodeRaw, dev, hp, st)) != ZCCL_OK) return rc;
    }
    if ((rc = flush_encode(c, b, kEncodeRaw, dev, hp, st)) != ZCCL_OK) return rc;

    if (N > 1) {   // tree forwarding: chunk ch moves to holder h + d in every round whose distance d it is beyond
        int top = 1;
        while (2 * top < N) top *= 2;
        ChainBatch cb{};
        cb.slots = c->arena; cb.sizes = g_sz; cb.slot_bytes = slot; cb.N = N; cb.hops = -1; cb.count = 0;
        for (int ch = 1; ch < N; ++ch) {
            ChainJob& j = cb.job[cb.count++];
            j.src0 = (const uint32_t*)gslot(0, ch); j.bytes = own_sz + ch; j.first_rank = 0; j.chunk = ch;
            j.path = 0; j.hops = 0;
            int h = 0;
            for (int d = top; d >= 1; d /= 2)
                if (ch >= h + d) { h += d; j.path |= (unsigned long long)h << (8 * j.hops); ++j.hops; }
        }
        if ((rc = cuda_rc(launch_copy_chain(cb, c->ws, c->sm_count, st))) != ZCCL_OK) return rc;
    }
    {   // the root keeps its own chunk as it is
        CopyBatcher cb;
        cb.add_fixed(root, recv[0], sizeof(float) * n);
        if ((rc = flush_copy(c, cb, st)) != ZCCL_OK) return rc;
    }
    for (int r = 1; r < N; ++r) {
        Job j{};
        j.in_c = (const uint32_t*)gslot(r, r); j.in_cap = slot; j.y = recv[r]; j.n = n;
        b.add(j, tiles_of(n));
        if (b.full() && (rc = flush_decode(c, b, st)) != ZCCL_OK) return rc;
    }
    return flush_decode(c, b, st);
}

int zccl_quality(zccl_ctx* c, const float* x, const float* y, size_t n, double* out, void* stream)
{
    if (!c || !x || !y || !out || n == 0 || n > c->max_elems) return ZCCL_E_ARG;
    if (((uintptr_t)x & 3u) || ((uintptr_t)y & 3u) || ((uintptr_t)out & 7u)) return ZCCL_E_ARG;
    return cuda_rc(launch_quality(x, y, n, out, c->quality_partials, c->quality_counter, c->sm_count, (cudaStream_t)stream));
}

static bool tile_ok(unsigned tile)
{
    return tile >= (unsigned)kGenericMinTile && tile <= (unsigned)kGenericMaxTile && tile % (unsigned)kBlock == 0;
}

size_t zccl_compress_bound_tiled(size_t n, unsigned tile)
{
    if (!tile_ok(tile)) return 0;
    const size_t nT = (n + tile - 1) / tile;
    size_t total = kHeaderBytes + 4 * nT;
    if (nT == 0) return total;
    const size_t full = nT - 1, bpt = tile / kBlock;
    total += full * (4 + ((bpt + 3) & ~(size_t)3) + bpt * 128);
    const size_t nb = (n - full * tile + kBlock - 1) / kBlock;
    total += 4 + ((nb + 3) & ~(size_t)3) + nb * 128;
    return total;
}

int zccl_compress_tiled(zccl_ctx* c, const float* x, size_t n, int eb_mode, float eb, unsigned tile,
                        void* out, size_t out_capacity, size_t* out_bytes, void* stream)
{
    if (!c || (!x && n) || !out || !out_bytes || !eb_ok(eb_mode, eb) || n > c->max_elems || !tile_ok(tile)) return ZCCL_E_ARG;
    if (((uintptr_t)x & 3u) || ((uintptr_t)out & 3u)) return ZCCL_E_ARG;
    const size_t nT = (n + tile - 1) / tile;
    if (nT > c->gen_tiles) return ZCCL_E_ARG;
    if (out_capacity < kHeaderBytes + 4 * nT) return ZCCL_E_CAPACITY;
    cudaStream_t st = (cudaStream_t)stream;
    Params hp{};
    bool dev = false;
    RangeList rl;
    rl.x.push_back(x); rl.n.push_back(n);
    int rc = resolve_bound(c, rl, eb_mode, eb, hp, dev, st);
    if (rc != ZCCL_OK) return rc;
    return cuda_rc(launch_generic_encode(x, n, tile, hp, dev, c->gen_sizes, c->gen_sizes + c->gen_tiles, (uint32_t*)out,
                                         out_capacity, out_bytes, c->ws, c->sm_count, st));
}

int zccl_compress_f64(zccl_ctx* c, const double* x, size_t n, int eb_mode, double eb, void* out, size_t out_capacity,
                      size_t* out_bytes, void* stream)
{
    if (!c || (!x && n) || !out || !out_bytes || n > c->max_elems) return ZCCL_E_ARG;
    if ((eb_mode != ZCCL_EB_ABS && eb_mode != ZCCL_EB_REL) || !(eb > 0.0) || !std::isfinite(eb)) return ZCCL_E_ARG;
    if (((uintptr_t)x & 7u) || ((uintptr_t)out & 3u)) return ZCCL_E_ARG;
    const size_t nT = tiles_of(n);
    if (nT > c->gen_tiles) return ZCCL_E_ARG;
    if (out_capacity < kHeaderBytes + 4 * nT) return ZCCL_E_CAPACITY;
    cudaStream_t st = (cudaStream_t)stream;
    ParamsF64 hp{0.0, 1.0, 1.0, 1};
    bool dev = false;
    if (eb_mode == ZCCL_EB_REL) {
        if (n == 0) return ZCCL_E_DEGENERATE;
        if (launch_range_f64(x, n, eb, c->ws, c->sm_count, st) != cudaSuccess) return ZCCL_E_CUDA;
        dev = true;
    } else {
        volatile double ebq = eb * (1.0 - 9.5367431640625e-07);   // 1 - 2^-20: one IEEE operation each, as on the device
        volatile double s = ebq * 2.0;
        if (!(s > 0.0) || !std::isfinite((double)s)) return ZCCL_E_DEGENERATE;
        volatile double r = 1.0 / s;
        if (!std::isfinite((double)r)) return ZCCL_E_DEGENERATE;
        hp.eb_abs = eb; hp.s = s; hp.r = r;
    }
    return cuda_rc(launch_encode_f64(x, n, hp, dev, c->gen_sizes, c->gen_sizes + c->gen_tiles, (uint32_t*)out, out_capacity, out_bytes,
                                     c->ws, c->sm_count, st));
}

int zccl_decompress_f64(zccl_ctx* c, const void* in, size_t in_bytes_max, double* y, size_t y_capacity_elems, void* stream)
{
    if (!c || !in || (!y && y_capacity_elems)) return ZCCL_E_ARG;
    if (((uintptr_t)in & 3u) || ((uintptr_t)y & 7u)) return ZCCL_E_ARG;
    if (in_bytes_max < (size_t)kHeaderBytes) return ZCCL_E_CAPACITY;
    return cuda_rc(launch_decode_f64((const uint32_t*)in, in_bytes_max, y, y_capacity_elems, c->ws, c->sm_count, (cudaStream_t)stream));
}

int zccl_decompress_tiled(zccl_ctx* c, const void* in, size_t in_bytes_max, unsigned tile, float* y, size_t y_capacity_elems,
                          void* stream)
{
    if (!c || !in || (!y && y_capacity_elems) || !tile_ok(tile)) return ZCCL_E_ARG;
    if (((uintptr_t)in & 3u) || ((uintptr_t)y & 3u)) return ZCCL_E_ARG;
    if (in_bytes_max < (size_t)kHeaderBytes) return ZCCL_E_CAPACITY;
    return cuda_rc(launch_generic_decode((const uint32_t*)in, in_bytes_max, tile, y, y_capacity_elems, c->ws, c->sm_count,
                                         (cudaStream_t)stream));
}

int zccl_stream_stats(zccl_ctx* c, const void* in, size_t in_bytes_max, unsigned long long* hist, void* stream)
{
    if (!c || !in || !hist || ((uintptr_t)in & 3u) || ((uintptr_t)hist & 7u)) return ZCCL_E_ARG;
    if (in_bytes_max < (size_t)kHeaderBytes) return ZCCL_E_CAPACITY;
    cudaStream_t st = (cudaStream_t)stream;
    if (cudaMemsetAsync(hist, 0, sizeof(unsigned long long) * 33, st) != cudaSuccess) return ZCCL_E_CUDA;
    return cuda_rc(launch_stream_stats((const uint32_t*)in, in_bytes_max, hist, c->ws, c->sm_count, st));
}

int zccl_range(zccl_ctx* c, const float* x, size_t n, float* minmax, void* stream)
{
    if (!c || (!x && n) || !minmax || n > c->max_elems) return ZCCL_E_ARG;
    if (((uintptr_t)x & 3u) || ((uintptr_t)minmax & 3u)) return ZCCL_E_ARG;
    cudaStream_t st = (cudaStream_t)stream;
    RangeBatch rb{};
    rb.x[0] = x; rb.n[0] = n; rb.count = 1;
    rb.finish = kRangeExport;
    rb.out = minmax;
    return cuda_rc(launch_range(rb, c->ws, c->sm_count, st));
}

int zccl_resolve_range_host(float mn, float mx, float eb_rel, float* eb_abs, float* step, float* reciprocal)
{
    if (!(eb_rel > 0.0f) || !std::isfinite(eb_rel)) return ZCCL_E_ARG;
    volatile float range = mx - mn;            // volatile: one IEEE fp32 operation each, as on the device
    if (!(mn <= mx) || !((float)range > 0.0f) || !std::isfinite((float)range)) return ZCCL_E_DEGENERATE;
    volatile float ea = eb_rel * range;
    Params p;
    const int rc = resolve_abs_host(ea, p);
    if (rc != ZCCL_OK) return rc;
    if (eb_abs) *eb_abs = ea;
    if (step) *step = p.s;
    if (reciprocal) *reciprocal = p.r;
    return ZCCL_OK;
}

int zccl_resolve_range(zccl_ctx* c, const float* minmax, float eb_rel, float* eb_abs_out, void* stream)
{
    if (!c || !minmax || !(eb_rel > 0.0f) || !std::isfinite(eb_rel)) return ZCCL_E_ARG;
    if (((uintptr_t)minmax & 3u) || ((uintptr_t)eb_abs_out & 3u)) return ZCCL_E_ARG;
    return cuda_rc(launch_resolve_range(minmax, eb_rel, c->ws, eb_abs_out, (cudaStream_t)stream));
}

int zccl_scale(zccl_ctx* c, float* y, size_t n, float divisor, void* stream)
{
    if (!c || (!y && n) || ((uintptr_t)y & 3u) || !(divisor > 0.0f) || !std::isfinite(divisor)) return ZCCL_E_ARG;
    if (n == 0) return ZCCL_OK;
    ScaleBatch sb{};
    sb.y[0] = y; sb.n = n; sb.divisor = divisor; sb.count = 1;
    return cuda_rc(launch_scale(sb, c->sm_count, (cudaStream_t)stream));
}

int zccl_sim_sizes(zccl_ctx* c, size_t* sizes, int capacity, void* stream)
{
    if (!c || !sizes || capacity < 0) return ZCCL_E_ARG;
    cudaStream_t st = (cudaStream_t)stream;
    const int cnt = c->sim_sizes_count < capacity ? c->sim_sizes_count : capacity;
    if (cnt > 0 && cudaMemcpyAsync(sizes, c->sim_sizes, sizeof(size_t) * (size_t)cnt, cudaMemcpyDeviceToHost, st) != cudaSuccess)
        return ZCCL_E_CUDA;
    if (cudaStreamSynchronize(st) != cudaSuccess) return ZCCL_E_CUDA;
    return c->sim_sizes_count;
}

int zccl_compress_host(zccl_ctx* c, const float* x_host, size_t n, int eb_mode, float eb,
                       void* out_host, size_t out_capacity, size_t* out_bytes_host, void* stream)
{
    if (!c || (!x_host && n) || !out_host || !out_bytes_host || n > c->max_elems) return ZCCL_E_ARG;
    cudaStream_t st = (cudaStream_t)stream;
    if (n && cudaMemcpyAsync(c->stage_x, x_host, sizeof(float) * n, cudaMemcpyHostToDevice, st) != cudaSuccess) return ZCCL_E_CUDA;
    int rc = zccl_compress(c, c->stage_x, n, eb_mode, eb, c->stage_c, c->stage_c_cap, c->stage_bytes, stream);
    if (rc != ZCCL_OK) return rc;
    if (cudaMemcpyAsync(out_bytes_host, c->stage_bytes, sizeof(size_t), cudaMemcpyDeviceToHost, st) != cudaSuccess) return ZCCL_E_CUDA;
    if (cudaStreamSynchronize(st) != cudaSuccess) return ZCCL_E_CUDA;
    const size_t nbytes = *out_bytes_host;
    if (nbytes > out_capacity) return ZCCL_E_CAPACITY;
    if (nbytes && cudaMemcpyAsync(out_host, c->stage_c, nbytes, cudaMemcpyDeviceToHost, st) != cudaSuccess) return ZCCL_E_CUDA;
    // the stream is in host memory when the call returns: zccl_decompress_host reads its header on the host
    if (cudaStreamSynchronize(st) != cudaSuccess) return ZCCL_E_CUDA;
    return ZCCL_OK;
}

int zccl_decompress_host(zccl_ctx* c, const void* in_host, size_t in_bytes, float* y_host, size_t y_capacity_elems, void* stream)
{
    if (!c || !in_host || (!y_host && y_capacity_elems) || in_bytes > c->stage_c_cap) return ZCCL_E_ARG;
    if (in_bytes < (size_t)kHeaderBytes) return ZCCL_E_CAPACITY;
    cudaStream_t st = (cudaStream_t)stream;
    unsigned long long n = 0;
    std::memcpy(&n, (const uint8_t*)in_host + 8, 8);
    if (n > c->max_elems || n > y_capacity_elems) return ZCCL_E_CAPACITY;
    if (cudaMemcpyAsync(c->stage_c, in_host, in_bytes, cudaMemcpyHostToDevice, st) != cudaSuccess) return ZCCL_E_CUDA;
    int rc = zccl_decompress(c, c->stage_c, in_bytes, c->stage_x, (size_t)n, stream);
    if (rc != ZCCL_OK) return rc;
    if (n && cudaMemcpyAsync(y_host, c->stage_x, sizeof(float) * (size_t)n, cudaMemcpyDeviceToHost, st) != cudaSuccess) return ZCCL_E_CUDA;
    return ZCCL_OK;
}

}  // extern "C"
