// Internal declarations shared by the kernel translation unit and the C boundary.  Not installed.
#pragma once
#include <cuda_runtime.h>
#include <stddef.h>
#include <stdint.h>

namespace zccl {

constexpr uint32_t kMagic = 0x314C435Au;    // 'Z','C','L','1'
constexpr uint32_t kVersion = 0x05000001u;  // version 1, dtype 0 (fp32), log2(block) = 5
constexpr uint32_t kVersionF64 = 0x05000101u;  // the same with dtype 1 (fp64): header words 4..5 hold the step as one binary64
constexpr int kHeaderBytes = 32;
constexpr int kHeaderWords = 8;
constexpr int kBlock = 32;                  // elements per block = warp width
constexpr int kTile = 4096;                 // elements per tile (Lorenzo restart unit, one index entry)
constexpr int kBlocksPerTile = kTile / kBlock;
constexpr int kThreads = 256;               // one CTA works on one tile at a time
constexpr int kWarps = kThreads / 32;
constexpr int kBlocksPerWarp = kBlocksPerTile / kWarps;   // 16 consecutive blocks per warp
constexpr int kGenericMinTile = 1024;       // tile sizes the plain kernels of zccl_generic.cu accept (multiples of 32)
constexpr int kGenericMaxTile = 8192;
// Chunk-operations per launch.  A stage of an 8-rank ring (8 jobs) fits one launch.  (With 64 the fused hop's 64 MiB
// launch was 1.6 us slower; decoding launches alone take 64, see kMaxDecodeJobs.)
constexpr int kMaxJobs = 32;

// Device status bits (zccl_status maps them to return codes).
enum : uint32_t {
    kStCapacity = 1u << 0,
    kStRange = 1u << 1,
    kStBadStream = 1u << 2,
    kStTimeout = 1u << 3,
    kStDegenerate = 1u << 4,
    kStPrecision = 1u << 5,
};

// Resolved bound (device resident when the mode is value-range relative).
struct Params {
    float eb_abs;
    float s;      // quantisation step
    float r;      // fl32(1 / s)
    int valid;    // 0: resolution failed (degenerate range); codec kernels then write nothing
};

// Resolved bound for binary64 input (device resident when the mode is value-range relative).
struct ParamsF64 {
    double eb_abs;
    double s;     // quantisation step: 2 * fl64(eb_abs * (1 - 2^-20))
    double r;     // fl64(1 / s)
    int valid;
};

// Scan / bookkeeping workspace owned by the context.
struct Workspace {
    unsigned long long* tile_state;  // one 64-bit {epoch:31 | inclusive:1 | words:32} per tile of a launch
    unsigned long long* group_state; // the same per group of 32 consecutive tiles of a job: group_slots(max_tiles) entries
    unsigned long long* group_acc;   // per group {tiles published:24 | their words:40}, zero between launches
    uint32_t* ticket;                // next tile to hand out
    uint32_t* done;                  // CTAs that have finished (the last one resets ticket/done, bumps epoch)
    uint32_t* epoch;                 // launch counter that validates tile_state entries
    uint32_t* status;                // device status bits
    Params* params;                  // resolved bound for REL mode
    uint32_t* minmax;                // two ordered-int keys: running min and max
    ParamsF64* params64;             // the same two for binary64 input (null in the allocation-free workspace)
    unsigned long long* minmax64;
    // Two-step compression (encode rounds into fixed slots, then place): null where there is no room for it (the
    // allocation-free entry point), which then compresses in a single pass.
    uint32_t* slots;                 // per round of a launch (4 per tile): kRoundSlotWords words
    uint32_t* round_words;           // per round: its payload words
    int32_t* outliers;               // per tile: its first quantised value
    uint32_t max_tiles;
    uint32_t skip_publish;           // test hook: tile number whose size is never published (0xFFFFFFFF = off)
};

// A round's slot: the code-length bytes of its 32 blocks (8 words), then its payload at the largest code length.
constexpr int kRoundSlotWords = 8 + 32 * 32;

// Groups of 32 tiles never span jobs, so a launch needs at most one slot per 32 tiles plus one per job.
__host__ __device__ constexpr unsigned long long group_slots(unsigned long long max_tiles) { return max_tiles / 32 + kMaxJobs + 2; }

// One chunk-operation.  Encoding jobs (compress, fused hop) and decoding jobs share the struct.
struct Job {
    const float* x;         // compress: input; fused: uncompressed local operand (or nullptr)
    const uint32_t* in_c;   // decode / fused: compressed input stream
    const uint32_t* in_c2;  // fused, two-compressed form: second stream (or nullptr)
    uint32_t* out;          // encode: output stream
    size_t* out_bytes;      // encode: receives stream length
    float* y;               // decode: output; fused: optional uncompressed sum (or nullptr)
    unsigned long long n;           // elements (decode: capacity of y in elements)
    unsigned long long out_cap;     // encode: capacity of out in bytes
    unsigned long long in_cap;      // bytes readable at in_c
    unsigned long long in2_cap;     // bytes readable at in_c2
    uint32_t tile_begin;    // first global tile number of this job within the launch
    uint32_t flags;
};

template <int CAP>
struct JobBatchT {
    Job job[CAP];
    int count;
    uint32_t total_tiles;
};
using JobBatch = JobBatchT<kMaxJobs>;
// Decoding launches take twice as many: the 56 chunk decodes that end an 8-rank Allreduce or Allgather are one launch.
constexpr int kMaxDecodeJobs = 64;
using DecodeBatch = JobBatchT<kMaxDecodeJobs>;

struct CopyJob {
    const uint32_t* src;
    uint32_t* dst;
    const size_t* bytes;   // device-resident length (nullptr: the length is `fixed_bytes`)
    size_t* bytes_out;     // optional: where to record the length at the destination
    unsigned long long cap;
    unsigned long long fixed_bytes;
};
struct CopyBatch {
    CopyJob job[kMaxJobs];
    int count;
};

// All forwarding hops of a ring Allgather stage in one launch.  Chain c carries one compressed chunk from its
// first holder around the ring: hop h copies it from where hop h - 1 left it to the slot of rank
// (first_rank + h) mod N.  Slots are laid out regularly: rank r keeps chunk c at slots + (r * N + c) * slot_bytes
// and its length at sizes[r * N + c].
constexpr int kMaxChains = 64;
struct ChainJob {
    const uint32_t* src0;   // where the chunk is before the first hop
    const size_t* bytes;    // its device-resident length
    int first_rank;         // ring: receiver of the first hop (hop h goes to rank first_rank + h mod N)
    int chunk;
    unsigned long long path;   // tree: receiver of hop h in bits 8h .. 8h+7 (at most 8 hops)
    int hops;                  // tree: hops of this chain
};
struct ChainBatch {
    ChainJob job[kMaxChains];
    unsigned char* slots;
    size_t* sizes;
    unsigned long long slot_bytes;
    int N, hops, count;   // hops < 0: every chain follows its own path
};

// Average: every rank's result divided by the number of ranks (one fp32 division per element), grid.y = buffer.
struct ScaleBatch {
    float* y[kMaxJobs];
    unsigned long long n;
    float divisor;
    int count;
};

// What the last CTA of a range launch does with the collected minimum and maximum.
enum RangeFinish { kRangeOnly = 0, kRangeResolve = 1, kRangeExport = 2 };

struct RangeBatch {
    const float* x[kMaxJobs];
    unsigned long long n[kMaxJobs];
    int count;
    int finish;     // RangeFinish
    float eb;       // kRangeResolve: the relative bound
    float* out;     // kRangeExport: receives (min, max)
};

enum EncodeMode { kEncodeRaw = 0, kEncodeFused = 1 };

// Launchers (defined next to the kernels).
cudaError_t launch_range(const RangeBatch& rb, const Workspace& ws, int sm_count, cudaStream_t st);
cudaError_t launch_encode(const JobBatch& jb, EncodeMode mode, const Workspace& ws, bool device_params,
                          Params host_params, int sm_count, cudaStream_t st);
cudaError_t launch_encode_lanes(const JobBatch& jb, const Workspace& ws, bool device_params, Params host_params, int sm_count,
                                cudaStream_t st);
cudaError_t launch_hop_lanes(const JobBatch& jb, const Workspace& ws, int sm_count, cudaStream_t st);
cudaError_t launch_decode_lanes(const JobBatch& jb, const Workspace& ws, int sm_count, cudaStream_t st);
cudaError_t launch_decode(const JobBatch& jb, const Workspace& ws, int sm_count, cudaStream_t st);
cudaError_t launch_decode_wide(const DecodeBatch& jb, const Workspace& ws, int sm_count, cudaStream_t st);
cudaError_t launch_decode_lanes_wide(const DecodeBatch& jb, const Workspace& ws, int sm_count, cudaStream_t st);
cudaError_t launch_scale(const ScaleBatch& sb, int sm_count, cudaStream_t st);
cudaError_t launch_resolve_range(const float* minmax, float eb, const Workspace& ws, float* eb_abs_out, cudaStream_t st);
cudaError_t launch_generic_encode(const float* x, unsigned long long n, uint32_t T, Params hp, bool device_params, uint32_t* sizes,
                                  uint32_t* go, uint32_t* out, unsigned long long out_cap, size_t* out_bytes, const Workspace& ws,
                                  int sm_count, cudaStream_t st);
cudaError_t launch_generic_decode(const uint32_t* in, unsigned long long cap_bytes, uint32_t T, float* y, unsigned long long y_cap,
                                  const Workspace& ws, int sm_count, cudaStream_t st);
cudaError_t launch_encode_f64(const double* x, unsigned long long n, ParamsF64 hp, bool device_params, uint32_t* sizes, uint32_t* go,
                              uint32_t* out, unsigned long long out_cap, size_t* out_bytes, const Workspace& ws, int sm_count, cudaStream_t st);
cudaError_t launch_decode_f64(const uint32_t* in, unsigned long long cap_bytes, double* y, unsigned long long y_cap, const Workspace& ws,
                              int sm_count, cudaStream_t st);
// binary32 at another tile size on the tuned kernels (tiled_lanes_fit: the context's slots cover the launch)
bool tiled_lanes_fit(unsigned long long n, uint32_t T, const Workspace& ws);
cudaError_t launch_encode_tiled_lanes(const float* x, unsigned long long n, uint32_t T, Params hp, bool device_params, uint32_t* out,
                                      unsigned long long out_cap, size_t* out_bytes, const Workspace& ws, int sm_count, cudaStream_t st);
cudaError_t launch_decode_tiled_lanes(const uint32_t* in, unsigned long long cap_bytes, uint32_t T, float* y, unsigned long long y_cap,
                                      const Workspace& ws, int sm_count, cudaStream_t st);
// binary64 on the tuned kernels (a context with round slots)
cudaError_t launch_encode_f64_lanes(const double* x, unsigned long long n, ParamsF64 hp, bool device_params, uint32_t* out,
                                    unsigned long long out_cap, size_t* out_bytes, const Workspace& ws, int sm_count, cudaStream_t st);
cudaError_t launch_decode_f64_lanes(const uint32_t* in, unsigned long long cap_bytes, double* y, unsigned long long y_cap, const Workspace& ws,
                                    int sm_count, cudaStream_t st);
cudaError_t launch_range_f64(const double* x, unsigned long long n, double eb, const Workspace& ws, int sm_count, cudaStream_t st);
cudaError_t launch_stream_stats(const uint32_t* in, unsigned long long cap_bytes, unsigned long long* hist, const Workspace& ws,
                                int sm_count, cudaStream_t st);
cudaError_t launch_copy(const CopyBatch& cb, const Workspace& ws, int sm_count, cudaStream_t st);
// quality metrics: `partials` holds 4 doubles per CTA of the launch (at most kQualityCtas), `counter` one word that
// is zero between launches
constexpr int kQualityCtas = 1024;
cudaError_t launch_quality(const float* x, const float* y, unsigned long long n, double* out, double* partials,
                           uint32_t* counter, int sm_count, cudaStream_t st);
// extra: plain copies that ride along in the same launch (or nullptr)
cudaError_t launch_copy_chain(const ChainBatch& cb, const Workspace& ws, int sm_count, cudaStream_t st, const CopyBatch* extra = nullptr);
unsigned long long launch_count();
void count_launches(unsigned k);   // adds to the process-wide count of kernels this library has launched

}  // namespace zccl
