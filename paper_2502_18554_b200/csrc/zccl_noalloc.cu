// zccl_compress_noalloc: the compressor for callers that must not allocate device memory.
//
// Some callers cannot call cudaMalloc at all: code running inside a CUDA-graph capture or a stream-ordered region
// where an allocation would synchronise or be illegal, plug-ins that are handed a fixed memory budget by their host
// application, and teardown / out-of-memory handlers that run when the allocator is exhausted or no longer usable.
// zccl_ctx_create allocates the placement-scan workspace; this entry point keeps an equivalent workspace in a
// file-scope __device__ array instead, so it needs no context and never allocates or frees.
//
// The array's name is only a host-side stand-in in host code, not a device address: its address on the current
// device is looked up once per device with cudaGetSymbolAddress (checked) and that pointer is what the kernels get.
#include "../../include/zccl.h"
#include "zccl_internal.h"

#include <cmath>
#include <mutex>

using namespace zccl;

namespace {

constexpr size_t kMaxElems = (size_t)ZCCL_NOALLOC_MAX_ELEMS;
constexpr size_t kMaxTiles = kMaxElems / kTile + 1;
constexpr size_t kStateBytes = ((kMaxTiles + 2 * (size_t)group_slots(kMaxTiles)) * 8 + 255) / 256 * 256;
constexpr size_t kScratchBytes = kStateBytes;

// Scratch shared by every call on a device (about 140 KiB of scan states plus a block of counters, held by each GPU
// that loads the library until exit).  The counter block carries its starting values in the module image (the scan
// states are validated against a launch counter that starts at 1), so no call ever has to initialise anything and
// calls from any thread on any stream find the scratch ready.
static __device__ __align__(256) unsigned char g_noalloc_scratch[kScratchBytes];
static __device__ __align__(256) uint32_t g_noalloc_ctrl[64] = {0u /* ticket */, 0u /* done */, 1u /* launch counter */};

struct DeviceSetup {
    bool ready = false;
    unsigned char* base = nullptr;   // device address of g_noalloc_scratch on that device
    uint32_t* ctrl = nullptr;        // and of g_noalloc_ctrl
    int sm_count = 0;
};
constexpr int kMaxDevices = 64;
DeviceSetup g_setup[kMaxDevices];
std::mutex g_setup_mu;

// Runs after the encoder on the same stream: a device-side error turns the reported length into 0, and the shared
// status word is cleared so that the next call starts clean.
__global__ void noalloc_finalize_kernel(uint32_t* status, size_t* out_bytes)
{
    const uint32_t bits = *status;
    if (bits & (kStCapacity | kStRange | kStBadStream | kStTimeout | kStDegenerate)) *out_bytes = 0;
    *status = 0;
}

Workspace workspace_at(unsigned char* base, uint32_t* sm)
{
    Workspace ws{};
    ws.tile_state = reinterpret_cast<unsigned long long*>(base);
    ws.group_state = ws.tile_state + kMaxTiles;
    ws.group_acc = ws.group_state + group_slots(kMaxTiles);
    ws.ticket = sm + 0;
    ws.done = sm + 1;
    ws.epoch = sm + 2;
    ws.status = sm + 3;
    ws.params = reinterpret_cast<Params*>(sm + 4);
    ws.minmax = sm + 8;
    ws.params64 = nullptr; ws.minmax64 = nullptr;
    ws.slots = nullptr; ws.round_words = nullptr; ws.outliers = nullptr;
    ws.max_tiles = (uint32_t)kMaxTiles;
    ws.skip_publish = 0xFFFFFFFFu;
    return ws;
}

// First call on a device, with that device current: resolve the arrays' device addresses (host-side look-ups: nothing
// is enqueued, so there is nothing for a concurrent caller on another stream to wait for).
int setup_current_device(DeviceSetup** out)
{
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess) return ZCCL_E_CUDA;
    if (dev < 0 || dev >= kMaxDevices) return ZCCL_E_ARG;
    std::lock_guard<std::mutex> lock(g_setup_mu);
    DeviceSetup& s = g_setup[dev];
    if (!s.ready) {
        void* ptr = nullptr;
        void* ctrl = nullptr;
        if (cudaGetSymbolAddress(&ptr, g_noalloc_scratch) != cudaSuccess || ptr == nullptr) return ZCCL_E_CUDA;
        if (cudaGetSymbolAddress(&ctrl, g_noalloc_ctrl) != cudaSuccess || ctrl == nullptr) return ZCCL_E_CUDA;
        int sms = 0;
        if (cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess || sms <= 0) return ZCCL_E_CUDA;
        s.base = static_cast<unsigned char*>(ptr);
        s.ctrl = static_cast<uint32_t*>(ctrl);
        s.sm_count = sms;
        s.ready = true;
    }
    *out = &s;
    return ZCCL_OK;
}

}  // namespace

extern "C" int zccl_compress_noalloc(const float* x, size_t n, float eb_abs, void* out, size_t out_capacity,
                                     size_t* out_bytes, void* stream)
{
    if (!out || !out_bytes || (!x && n) || !(eb_abs > 0.0f) || !std::isfinite(eb_abs)) return ZCCL_E_ARG;
    if (((uintptr_t)out & 3u) || ((uintptr_t)x & 3u)) return ZCCL_E_ARG;
    if (n > kMaxElems) return ZCCL_E_TOO_LARGE;
    const size_t nT = (n + kTile - 1) / kTile;
    if (out_capacity < (size_t)kHeaderBytes + 4 * nT) return ZCCL_E_CAPACITY;

    // eb_abs -> step and reciprocal with the same IEEE operations as everywhere else
    volatile float ebq = eb_abs * 0.984375f;
    volatile float s = ebq * 2.0f;
    if (!(s > 0.0f) || !std::isfinite((float)s)) return ZCCL_E_DEGENERATE;
    volatile float r = 1.0f / s;
    if (!std::isfinite((float)r)) return ZCCL_E_DEGENERATE;
    Params hp;
    hp.eb_abs = eb_abs; hp.s = s; hp.r = r; hp.valid = 1;

    cudaStream_t st = (cudaStream_t)stream;
    DeviceSetup* dev = nullptr;
    const int rc = setup_current_device(&dev);
    if (rc != ZCCL_OK) return rc;
    const Workspace ws = workspace_at(dev->base, dev->ctrl);

    JobBatch jb{};
    jb.count = 1;
    Job& j = jb.job[0];
    j.x = x; j.out = (uint32_t*)out; j.out_bytes = out_bytes; j.n = n; j.out_cap = out_capacity; j.tile_begin = 0;
    jb.total_tiles = (uint32_t)(nT ? nT : 1);
    if (launch_encode(jb, kEncodeRaw, ws, false, hp, dev->sm_count, st) != cudaSuccess) return ZCCL_E_CUDA;
    count_launches(1);
    noalloc_finalize_kernel<<<1, 1, 0, st>>>(ws.status, out_bytes);
    return cudaGetLastError() == cudaSuccess ? ZCCL_OK : ZCCL_E_CUDA;
}
