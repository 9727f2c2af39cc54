// dnns_magnitude_threshold_static: the k-th-magnitude threshold of ONE weight tensor with all of
// its scratch memory inside this library instead of a caller-provided workspace.
//
// Who this is for: code that runs where device memory cannot be allocated - a plug-in called
// inside someone else's memory-planned inference or training step, a callback that runs while
// the host framework's allocator is locked, or a process whose memory budget was handed out in
// full at start-up.  Such a caller owns the weights and the 32-byte result record and nothing
// else; it cannot provide the few hundred kilobytes of histograms and tables that the plan-based
// entry point keeps in its workspace.
//
// The scratch is the file-scope array below.  It is part of the library image: every GPU that
// loads the library holds these ~0.6 MB until the process exits.  Host code must not pass the
// array's name to a kernel (on the host that name is only a stand-in for the symbol); the device
// address is obtained once per device with cudaGetSymbolAddress and handed to the kernels.
#include <atomic>
#include <mutex>

#include "dnns_internal.cuh"

namespace {

using namespace dnns;

constexpr uint64_t kMaxNumel = DNNS_STATIC_MAX_NUMEL;
constexpr uint32_t kMaxTiles = (uint32_t)(kMaxNumel * 4 / kTileBytes);  // fp32 is the wider case

// Byte offsets inside the scratch array (every section 256-byte aligned).
constexpr size_t kOffTensor = 0;                                  // TensorDesc[1]
constexpr size_t kOffSeg = 256;                                   // SegDesc[1]
constexpr size_t kOffK = 512;                                     // uint64 k
constexpr size_t kOffSel = 768;                                   // SelectState[1]
constexpr size_t kOffSplit = 896;                                 // TieSplit[1]
constexpr size_t kOffBitmap = 1024;                               // kBitmapWords words
constexpr size_t kOffTileTensor = kOffBitmap + 4 * kBitmapWords;  // kMaxTiles words, always zero (tensor 0)
constexpr size_t kOffTiePrefix = kOffTileTensor + 4 * (size_t)kMaxTiles;
// --- everything from here on is cleared at the start of every call ---
constexpr size_t kOffClear = kOffTiePrefix + 4 * (size_t)kMaxTiles;
constexpr size_t kOffAnyNeed = kOffClear;
constexpr size_t kOffNeed = kOffAnyNeed + 256;
constexpr size_t kOffTieBitmap = kOffNeed + 256;
constexpr size_t kOffTileTies = kOffTieBitmap + 4 * kBitmapWords;
constexpr size_t kOffHist1 = kOffTileTies + 4 * (size_t)kMaxTiles;
constexpr size_t kOffHist2 = kOffHist1 + 4 * (size_t)kHistBins;
constexpr size_t kScratchBytes = kOffHist2 + 4 * (size_t)kLowBins;

static __device__ __align__(256) unsigned char g_static_scratch[kScratchBytes];

constexpr int kMaxDevices = 64;
std::mutex g_mutex;
std::atomic<unsigned char*> g_scratch_ptr[kMaxDevices];  // device address of the array, per device ordinal
int g_n_sm[kMaxDevices] = {};                            // written before the pointer is published

// One-time set-up on the current device: resolve the device address of the scratch array and raise the
// shared-memory limit of the histogram kernel.  (A __device__ array without an initialiser starts as zeros, which
// is what the constant sections of the scratch - the tile -> tensor table - rely on.)  Loading the library's
// device code, which the first CUDA call of a process into this library triggers, happens here too.
dnns_status setup_device(int dev) {
    if (g_scratch_ptr[dev].load(std::memory_order_acquire)) return DNNS_OK;
    std::lock_guard<std::mutex> lock(g_mutex);
    if (g_scratch_ptr[dev].load(std::memory_order_relaxed)) return DNNS_OK;
    unsigned char* p = nullptr;
    if (cudaGetSymbolAddress(reinterpret_cast<void**>(&p), g_static_scratch) != cudaSuccess || !p) return DNNS_ERR_CUDA;
    int n_sm = 0;
    if (cudaDeviceGetAttribute(&n_sm, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess) return DNNS_ERR_CUDA;
    if (init_kernel_attributes() != cudaSuccess) return DNNS_ERR_CUDA;
    g_n_sm[dev] = n_sm;
    g_scratch_ptr[dev].store(p, std::memory_order_release);
    return DNNS_OK;
}

// The descriptors of the call travel as kernel arguments (copied when the launch is enqueued - or captured - not
// when it runs) and are stored into the scratch by one thread.
__global__ void k_static_descriptors(TensorDesc td, SegDesc sd, TensorDesc* td_out, SegDesc* sd_out) {
    *td_out = td;
    *sd_out = sd;
}

}  // namespace

extern "C" dnns_status dnns_magnitude_threshold_static(const void* weights_dev, int32_t dtype, uint64_t numel,
                                                       uint64_t k, dnns_threshold* thr_dev, void* stream) {
    if (!weights_dev || !thr_dev || numel == 0) return DNNS_ERR_INVALID_ARG;
    if (reinterpret_cast<uintptr_t>(weights_dev) & 15) return DNNS_ERR_INVALID_ARG;
    if (dtype != DNNS_F32 && dtype != DNNS_BF16) return DNNS_ERR_UNSUPPORTED;
    if (numel > kMaxNumel) return DNNS_ERR_STATIC_LIMIT;
    if (k > numel) return DNNS_ERR_INVALID_ARG;
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess) return DNNS_ERR_CUDA;
    if (dev < 0 || dev >= kMaxDevices) return DNNS_ERR_UNSUPPORTED;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    if (!g_scratch_ptr[dev].load(std::memory_order_acquire)) {
        // the first call on a device resolves the array's address: not something a stream capture can record
        cudaStreamCaptureStatus cap = cudaStreamCaptureStatusNone;
        if (cudaStreamIsCapturing(st, &cap) != cudaSuccess) return DNNS_ERR_CUDA;
        if (cap != cudaStreamCaptureStatusNone) return DNNS_ERR_UNSUPPORTED;
    }
    const dnns_status s = setup_device(dev);
    if (s != DNNS_OK) return s;
    unsigned char* base = g_scratch_ptr[dev].load(std::memory_order_acquire);

    const uint32_t elem_bytes = dtype == DNNS_F32 ? 4 : 2;
    const uint32_t n_tiles = (uint32_t)((numel * elem_bytes + kTileBytes - 1) / kTileBytes);

    // descriptors of the one tensor and its one ranking segment
    TensorDesc td{};
    td.src = weights_dev;
    td.numel = (uint32_t)numel;
    td.O = 1, td.I = (int32_t)numel, td.KK = 1, td.S = 1;
    td.out_group = td.in_group = 0;
    td.seg = 0, td.bn = -1;
    td.tile0 = 0, td.n_tiles = n_tiles;
    const SegDesc sd{0, n_tiles, numel};

    // what must start at zero: histograms, tie tables and flags of the previous call
    if (cudaMemsetAsync(base + kOffClear, 0, kScratchBytes - kOffClear, st) != cudaSuccess) return DNNS_ERR_CUDA;
    k_static_descriptors<<<1, 1, 0, st>>>(td, sd, reinterpret_cast<TensorDesc*>(base + kOffTensor),
                                          reinterpret_cast<SegDesc*>(base + kOffSeg));
    if (cudaGetLastError() != cudaSuccess) return DNNS_ERR_CUDA;

    Tables tb{};
    tb.tensors = reinterpret_cast<const TensorDesc*>(base + kOffTensor);
    tb.segs = reinterpret_cast<const SegDesc*>(base + kOffSeg);
    tb.tile_tensor = reinterpret_cast<const uint32_t*>(base + kOffTileTensor);
    tb.n_tensors = 1, tb.n_segs = 1, tb.n_tiles = n_tiles;
    tb.tile_elems = kTileBytes / elem_bytes;
    tb.dtype = dtype;
    ThresholdWs ws{};
    ws.k_dev = reinterpret_cast<uint64_t*>(base + kOffK);
    ws.hist1 = reinterpret_cast<uint32_t*>(base + kOffHist1);
    ws.hist2 = reinterpret_cast<uint32_t*>(base + kOffHist2);
    ws.bitmap = reinterpret_cast<uint32_t*>(base + kOffBitmap);
    ws.tie_bitmap = reinterpret_cast<uint32_t*>(base + kOffTieBitmap);
    ws.sel = reinterpret_cast<SelectState*>(base + kOffSel);
    ws.need = reinterpret_cast<uint32_t*>(base + kOffNeed);
    ws.any_need = reinterpret_cast<uint32_t*>(base + kOffAnyNeed);
    ws.tile_ties = reinterpret_cast<uint32_t*>(base + kOffTileTies);
    ws.tie_prefix = reinterpret_cast<uint32_t*>(base + kOffTiePrefix);
    ws.split = reinterpret_cast<TieSplit*>(base + kOffSplit);
    return launch_threshold(tb, ws, 1, &k, thr_dev, g_n_sm[dev], st) < 0 ? DNNS_ERR_CUDA : DNNS_OK;
}
