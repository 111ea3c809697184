// Device-side helpers shared by the kernel translation units: scan-state words, mbarrier and bulk-copy wrappers,
// stream header parsing, job lookup, launch re-arming, and the host-side launch wrapper.  Not installed.
#pragma once
#include "zccl_internal.h"

#include <cstdlib>

namespace zccl {
namespace {

constexpr unsigned kFull = 0xFFFFFFFFu;
constexpr int kSpinLimit = 1 << 20;            // polls of a scan state or an mbarrier before giving up
constexpr float kRoundMagic = 12582912.0f;     // 1.5 * 2^23: t + kRoundMagic has rint(t) in its low mantissa bits
constexpr uint32_t kRoundMagicBits = 0x4B400000u;
constexpr float kTwo23 = 8388608.0f;           // 2^23: |d| + 2^23 has the integer |d| in its mantissa
constexpr float kGuardExact = 8.796093e12f;    // 2^43: sum of squares below it => every |x r| < 2^21.5
constexpr float kGuardSmall = 1.0e9f;          // below 2^30: no |x r| can exceed 2^15

// ------------------------------------------------------------------------------------------------ small helpers

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

__device__ __forceinline__ uint32_t smem_u32(const void* p) { return (uint32_t)__cvta_generic_to_shared(p); }

__device__ __forceinline__ void mbar_init(unsigned long long* bar, uint32_t count)
{
    asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(smem_u32(bar)), "r"(count) : "memory");
}
__device__ __forceinline__ void mbar_expect_tx(unsigned long long* bar, uint32_t bytes)
{
    asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(smem_u32(bar)), "r"(bytes) : "memory");
}
__device__ __forceinline__ bool mbar_try_wait(unsigned long long* bar, uint32_t parity)
{
    uint32_t ok;
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\t"
        "selp.u32 %0, 1, 0, p;\n\t}"
        : "=r"(ok) : "r"(smem_u32(bar)), "r"(parity) : "memory");
    return ok != 0;
}
// Bounded wait for a bulk copy to land; false after kSpinLimit polls.
__device__ __forceinline__ bool mbar_wait(unsigned long long* bar, uint32_t parity)
{
    for (int it = 0; it < kSpinLimit; ++it)
        if (mbar_try_wait(bar, parity)) return true;
    return false;
}
// 1-D bulk copy global -> this CTA's shared memory; addresses and size are multiples of 16 bytes.  The proxy
// fence orders earlier ordinary accesses to the destination before the copy engine's writes.
__device__ __forceinline__ void bulk_load(void* dst, const void* src, uint32_t bytes, unsigned long long* bar)
{
    asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
    asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];"
                 ::"r"(smem_u32(dst)), "l"(src), "r"(bytes), "r"(smem_u32(bar)) : "memory");
}

// Asks for a 16-byte-aligned range of global memory to be brought into L2 (no destination, nothing to wait for).
__device__ __forceinline__ void bulk_prefetch_l2(const void* src, uint32_t bytes)
{
    asm volatile("cp.async.bulk.prefetch.L2.global [%0], %1;" ::"l"(src), "r"(bytes) : "memory");
}

__device__ __forceinline__ uint32_t prmt(uint32_t a, uint32_t b, uint32_t sel)
{
    uint32_t d;
    asm("prmt.b32 %0, %1, %2, %3;" : "=r"(d) : "r"(a), "r"(b), "r"(sel));
    return d;
}

// The job that owns tile number `ticket` of the launch: the last one whose first tile is not beyond it.
template <class JB>
__device__ __forceinline__ int find_job(const JB& jb, uint32_t ticket)
{
    int lo = 0, hi = jb.count;
#pragma unroll 1
    while (hi - lo > 1) {
        const int mid = (lo + hi) >> 1;
        if (jb.job[mid].tile_begin <= ticket) lo = mid;
        else hi = mid;
    }
    return lo;
}

// Programmatic dependent launch: every kernel of the library is launched with stream serialisation relaxed, so that
// its CTAs are dispatched while the kernel in front of it on the stream drains, and waits here, before it touches
// memory, until that kernel has completed and its writes are visible.  Only then does it let the kernel behind it
// start to launch, so at most one waiting grid is resident at a time.  Without the launch attribute both
// instructions do nothing.
__device__ __forceinline__ void pdl_enter()
{
    asm volatile("griddepcontrol.wait;" ::: "memory");
    asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
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

__device__ __forceinline__ void write_header(uint32_t* out, int tid, unsigned long long n, float eb_abs, float s, uint32_t nT)
{
    if (tid < kHeaderWords) {
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
        out[tid] = hv;
    }
}

__device__ __forceinline__ void finish_launch(const Workspace& ws, uint32_t epoch, int tid, uint32_t* tile_counter = nullptr,
                                              uint32_t groups_used = 0)
{
    __syncthreads();
    if (tid == 0) {
        __threadfence();
        const uint32_t prev = atomicAdd(ws.done, 1u);
        if (prev == gridDim.x - 1) {   // every CTA is done with the scan states: re-arm for the next launch
            *ws.done = 0;
            if (tile_counter) *tile_counter = 0;
            for (uint32_t g = 0; g < groups_used; ++g) ws.group_acc[g] = 0ull;   // the group accumulators of this launch
            uint32_t e = (epoch + 1u) & 0x7FFFFFFFu;
            if (e == 0) {   // the counter wraps (once in 2^31 launches): no state of an earlier launch may look current again
                for (uint32_t t = 0; t < ws.max_tiles; ++t) st_state(ws.tile_state + t, 0ull);
                for (uint32_t t = 0; t < (uint32_t)group_slots(ws.max_tiles); ++t) st_state(ws.group_state + t, 0ull);
                __threadfence();
                e = 1u;
            }
            *ws.epoch = e;
        }
    }
}

__device__ __forceinline__ void mbar_arrive(unsigned long long* bar)
{
    asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(smem_u32(bar)) : "memory");
}

inline bool pdl_enabled()
{
    static const bool on = [] { const char* e = getenv("ZCCL_PDL"); return !(e && e[0] == '0'); }();
    return on;
}

template <bool EARLY = true, class... KArgs, class... Args>
cudaError_t launch_k(void (*kernel)(KArgs...), dim3 grid, dim3 block, size_t smem, cudaStream_t st, Args&&... args)
{
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = grid;
    cfg.blockDim = block;
    cfg.dynamicSmemBytes = smem;
    cfg.stream = st;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = (EARLY && pdl_enabled()) ? 1 : 0;
    cfg.attrs = attr;
    cfg.numAttrs = 1;
    return cudaLaunchKernelEx(&cfg, kernel, static_cast<KArgs>(args)...);
}


}  // namespace
}  // namespace zccl
