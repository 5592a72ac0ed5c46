// gg_fit_noalloc: the moments + fit step for one segment without any allocation.
//
// Some callers may not allocate device memory when they need a fit: code that runs while a memory
// pool owns the whole device and forbids side allocations, a training step whose allocator is
// frozen so that addresses stay stable, or a plug-in that is handed buffers and a stream and
// nothing else.  gg_fit needs a context whose plan (tile tables and per-tile partial sums) lives
// in memory obtained with cudaMalloc on first use; this entry point keeps the same tables and
// partials in a fixed array that is part of the loaded library image instead.
//
// The array below is device memory that every GPU loading the library holds until the process
// exits (about 0.7 MB).  In host code its name is only a handle: the device address is looked up
// once per device with cudaGetSymbolAddress and that pointer is what the kernels receive.
#include <mutex>

#include "gg_internal.h"

namespace {

using namespace gg;

constexpr int kMaxTiles = 16384;                       // 16384 tiles x 16384 elements
constexpr int64_t kMaxLen = (int64_t)kMaxTiles * kTile;
constexpr int kMaxDevices = 64;

// Byte layout of the scratch array (every piece starts on a 256-byte boundary).
constexpr size_t kOffSegPtr = 0;                       // const void *[1]
constexpr size_t kOffSegLen = 256;                     // int64[1]
constexpr size_t kOffPrefix = 512;                     // int32[2]
constexpr size_t kOffHistId = 768;                     // int32[1]
constexpr size_t kOffTileSeg = 1024;                   // int32[kMaxTiles]
constexpr size_t kOffS1 = kOffTileSeg + sizeof(int32_t) * kMaxTiles;
constexpr size_t kOffS2 = kOffS1 + sizeof(double) * kMaxTiles;
constexpr size_t kOffPen = kOffS2 + sizeof(double) * kMaxTiles;
constexpr size_t kOffBad = kOffPen + sizeof(double) * kMaxTiles;
constexpr size_t kOffMin = kOffBad + sizeof(uint32_t) * kMaxTiles;
constexpr size_t kOffMax = kOffMin + sizeof(float) * kMaxTiles;
constexpr size_t kScratchBytes = kOffMax + sizeof(float) * kMaxTiles;

static __device__ __align__(256) unsigned char g_noalloc_scratch[kScratchBytes];

// Per-device state of the one-time set-up.
struct DeviceSlot {
    bool ready = false;
    bool arch_ok = false;
    unsigned char *scratch = nullptr;   // device address of g_noalloc_scratch on this device
};
DeviceSlot g_slots[kMaxDevices];
std::mutex g_slots_mutex;

// Writes the one-segment tile tables.  The array keeps whatever the previous call left, so all
// that this call reads before writing is rewritten here: the segment entry, the tile prefix and
// the owning-segment index (zero) of each tile in use.  The per-tile partials need no clearing:
// the moments kernel writes every slot of [0, n_tiles) before the fit kernel reads it.
__global__ void noalloc_setup_kernel(unsigned char *scratch, const void *x, int64_t len, int32_t n_tiles)
{
    const int i = blockIdx.x * blockDim.x + threadIdx.x;
    if (i == 0) {
        *reinterpret_cast<const void **>(scratch + kOffSegPtr) = x;
        *reinterpret_cast<int64_t *>(scratch + kOffSegLen) = len;
        reinterpret_cast<int32_t *>(scratch + kOffPrefix)[0] = 0;
        reinterpret_cast<int32_t *>(scratch + kOffPrefix)[1] = n_tiles;
        *reinterpret_cast<int32_t *>(scratch + kOffHistId) = 0;
    }
    if (i < n_tiles) reinterpret_cast<int32_t *>(scratch + kOffTileSeg)[i] = 0;
}

struct CurrentDevice {
    int prev = -1, want = -1;
    bool ok = true;
    explicit CurrentDevice(int dev) : want(dev)
    {
        if (cudaGetDevice(&prev) != cudaSuccess) { ok = false; prev = -1; return; }
        if (prev != dev && cudaSetDevice(dev) != cudaSuccess) ok = false;
    }
    ~CurrentDevice() { if (prev >= 0 && prev != want) cudaSetDevice(prev); }
};

}  // namespace

extern "C" {

int64_t gg_fit_noalloc_max_len(void) { return kMaxLen; }

gg_status gg_fit_noalloc(int device, const void *x, int64_t len, gg_dtype dtype, double *beta,
                         double *alpha, double *sum_abs, double *sum_sq, int64_t *count,
                         uint32_t *flags, void *stream)
{
    if (device < 0 || device >= kMaxDevices || !beta || !alpha || len < 0) return GG_ERR_INVALID_ARG;
    if (dtype != GG_F32 && dtype != GG_BF16) return GG_ERR_DTYPE;
    if (len > 0 && x == nullptr) return GG_ERR_INVALID_ARG;
    if (reinterpret_cast<uintptr_t>(x) % (dtype == GG_F32 ? 4 : 2) != 0) return GG_ERR_ALIGNMENT;
    if (len > kMaxLen) return GG_ERR_WORKSPACE;     // more tiles than the fixed array has slots for

    CurrentDevice cur(device);
    if (!cur.ok) { cudaGetLastError(); return GG_ERR_CUDA; }

    // One-time set-up on this device (with the device current): architecture check and the device
    // address of the scratch array.  Neither call allocates; both are illegal during stream
    // capture, which is why the first call on a device belongs before any capture.
    DeviceSlot slot;
    {
        std::lock_guard<std::mutex> lock(g_slots_mutex);
        DeviceSlot &s = g_slots[device];
        if (!s.ready) {
            int major = 0;
            cudaError_t e = cudaDeviceGetAttribute(&major, cudaDevAttrComputeCapabilityMajor, device);
            if (e != cudaSuccess) { cudaGetLastError(); return GG_ERR_CUDA; }
            s.arch_ok = major == 10;
            if (s.arch_ok) {
                void *p = nullptr;
                e = cudaGetSymbolAddress(&p, g_noalloc_scratch);
                if (e != cudaSuccess || p == nullptr) { cudaGetLastError(); return GG_ERR_CUDA; }
                s.scratch = static_cast<unsigned char *>(p);
            }
            s.ready = true;
        }
        slot = s;
    }
    if (!slot.arch_ok) return GG_ERR_ARCH;

    unsigned char *d = slot.scratch;
    const int32_t n_tiles = (int32_t)((len + kTile - 1) / kTile);
    cudaStream_t cs = static_cast<cudaStream_t>(stream);

    const int threads = 256;
    noalloc_setup_kernel<<<(n_tiles + threads) / threads, threads, 0, cs>>>(d, x, len, n_tiles);
    cudaError_t e = cudaGetLastError();
    if (e != cudaSuccess) return GG_ERR_CUDA;

    TileMap map{};
    map.seg_ptr = reinterpret_cast<const void *const *>(d + kOffSegPtr);
    map.grad_ptr = nullptr;
    map.seg_len = reinterpret_cast<const int64_t *>(d + kOffSegLen);
    map.tile_prefix = reinterpret_cast<const int32_t *>(d + kOffPrefix);
    map.tile_seg = reinterpret_cast<const int32_t *>(d + kOffTileSeg);
    map.hist_id = reinterpret_cast<const int32_t *>(d + kOffHistId);
    map.n_seg = 1;
    map.n_tiles = n_tiles;
    TileScratch part{};
    part.s1 = reinterpret_cast<double *>(d + kOffS1);
    part.s2 = reinterpret_cast<double *>(d + kOffS2);
    part.pen = reinterpret_cast<double *>(d + kOffPen);
    part.bad = reinterpret_cast<uint32_t *>(d + kOffBad);
    part.xmin = reinterpret_cast<float *>(d + kOffMin);
    part.xmax = reinterpret_cast<float *>(d + kOffMax);

    StreamArgs sa{};
    sa.map = map;
    sa.part = part;
    e = launch_stream(kMoments, dtype, GG_F32, false, sa, cs);
    if (e != cudaSuccess) { cudaGetLastError(); return GG_ERR_CUDA; }
    FitArgs fa{};
    fa.map = map;
    fa.part = part;
    fa.beta = beta; fa.alpha = alpha; fa.sum_abs = sum_abs; fa.sum_sq = sum_sq;
    fa.count = count; fa.flags = flags; fa.in_dtype_plus1 = (int)dtype + 1;
    e = launch_fit(fa, cs);
    if (e != cudaSuccess) { cudaGetLastError(); return GG_ERR_CUDA; }
    return GG_OK;
}

}  // extern "C"
