// gc_compress_noalloc: exact top-k compression of one tensor whose scratch memory is a fixed
// array inside the library image, for callers that must not allocate device memory.
#include "gc.h"

#include <mutex>

#include "gc_kernels.cuh"

using namespace gc;

namespace {

constexpr uint32_t kMaxN = GC_NOALLOC_MAX_N;
constexpr uint32_t kMaxTiles = (kMaxN + kTile - 1) / kTile;

// Layout of the fixed scratch (byte offsets, all multiples of 256 except the tail table).
constexpr size_t kOffSel = sizeof(WsHeader);
constexpr size_t kOffHist = 512;
constexpr size_t kOffState = kOffHist + sizeof(uint32_t) * kHistBins;
constexpr size_t kOffDesc = kOffState + sizeof(unsigned long long) * kMaxTiles;
constexpr size_t kScratchBytes = kOffDesc + 256;
static_assert(kOffSel + sizeof(TensorSel) <= kOffHist, "selection record fits before the histogram");
static_assert(kOffState % 256 == 0 && kOffDesc % 256 == 0, "aligned sections");

static_assert(kScratchBytes == 41728, "the documented size of the fixed scratch (about 41 KB) follows this layout");

// The scratch itself.  Every GPU that loads this library carries these 41,728 bytes until the
// process exits.  In host code this name is only a handle for cudaGetSymbolAddress; it is not
// a device address and must never be handed to a kernel directly.
static __device__ __align__(256) unsigned char g_noalloc_scratch[kScratchBytes];

struct PerDevice {
    void* scratch = nullptr;     // device address of g_noalloc_scratch on this device
    int grid_hist = 0, grid_compact = 0;
};
constexpr int kMaxDevices = 64;
PerDevice g_dev[kMaxDevices];
std::mutex g_dev_mutex;

// Clears every word that must start at zero (the array keeps the previous call's contents)
// and writes the one-tensor table the kernels read.
__global__ void k_noalloc_init(unsigned char* scratch, uint32_t n, uint32_t k, uint32_t ntiles) {
    const uint32_t tid = blockIdx.x * blockDim.x + threadIdx.x, nth = gridDim.x * blockDim.x;
    uint32_t* w = reinterpret_cast<uint32_t*>(scratch);
    const uint32_t ctrl_words = (uint32_t)((kOffState + sizeof(unsigned long long) * ntiles) / 4);
    for (uint32_t i = tid; i < ctrl_words; i += nth) w[i] = 0u;
    if (tid == 0) {
        TensorDesc d;
        d.off = 0; d.n = n; d.k = k; d.cap = k; d.out_off = 0; d.tile0 = 0; d.ntiles = ntiles; d.stride = 1;
        d.sstride = 0; d.srank = 0; d.stile0 = 0; d.nstiles = 0; d.group0 = 0; d.ngroups = 0;
        d.kind = kKindRegular; d.pad = 0;
        *reinterpret_cast<TensorDesc*>(scratch + kOffDesc) = d;
    }
}

__global__ void k_noalloc_finish(const unsigned char* scratch, int32_t* status_out) {
    if (status_out != nullptr) *status_out = reinterpret_cast<const WsHeader*>(scratch)->status;
}

// k = 0: nothing is sent, but the gradient still has to reach the error-feedback residual
// (r' = g + r, one rounding), exactly as the top-k rule leaves every unsent entry.
__global__ void __launch_bounds__(256) k_noalloc_fold_only(const float* __restrict__ g, float* __restrict__ r,
                                                           uint32_t n, int32_t* status_out) {
    const uint32_t nth = gridDim.x * blockDim.x;
    for (uint32_t i = blockIdx.x * blockDim.x + threadIdx.x; i < n; i += nth) r[i] = __fadd_rn(g[i], r[i]);
    if (status_out != nullptr && blockIdx.x == 0 && threadIdx.x == 0) *status_out = GC_OK;
}

}  // namespace

extern "C" int gc_compress_noalloc(const float* grad, float* residual, uint32_t n, uint32_t k,
                                   uint32_t* out_idx, float* out_val, int32_t* device_status,
                                   void* stream) {
    if (n > kMaxN) return GC_E_TOO_LARGE;        // beyond the fixed scratch: use gc_plan + gc_compress
    if (k > n) return GC_E_INVALID;
    cudaStream_t s = static_cast<cudaStream_t>(stream);
    if (n > 0 && (grad == nullptr || residual == nullptr)) return GC_E_INVALID;
    if (k > 0 && (out_idx == nullptr || out_val == nullptr)) return GC_E_INVALID;
    if ((reinterpret_cast<uintptr_t>(grad) & 15u) || (reinterpret_cast<uintptr_t>(residual) & 15u))
        return GC_E_INVALID;
    if (k == 0) {
        // nothing to select (and the scratch is not needed): fold only, or just report success
        if (n > 0 || device_status != nullptr) {
            const uint32_t blocks = n == 0 ? 1u : (n + 1023u) / 1024u;
            k_noalloc_fold_only<<<(int)(blocks < 1184u ? blocks : 1184u), 256, 0, s>>>(grad, residual, n, device_status);
            if (cudaGetLastError() != cudaSuccess) return GC_E_CUDA;
        }
        return GC_OK;
    }
    int dev = -1;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= kMaxDevices) {
        (void)cudaGetLastError();
        return GC_E_CUDA;
    }
    PerDevice pd;
    {
        // one-time set-up per device, with that device current: resolve the device address of
        // the scratch array and size the grids.  Nothing here allocates.
        std::lock_guard<std::mutex> lock(g_dev_mutex);
        if (g_dev[dev].scratch == nullptr) {
            void* ptr = nullptr;
            cudaError_t e = cudaGetSymbolAddress(&ptr, g_noalloc_scratch);
            int sms = 0, bh = 0, bc = 0;
            if (e == cudaSuccess) e = cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev);
            if (e == cudaSuccess)
                e = cudaOccupancyMaxActiveBlocksPerMultiprocessor(&bh, k_hist<0, SRC_FOLD>, kBlock, 0);
            if (e == cudaSuccess) e = cudaOccupancyMaxActiveBlocksPerMultiprocessor(&bc, k_compact, kBlock, 0);
            if (e != cudaSuccess || ptr == nullptr || sms < 1) {
                (void)cudaGetLastError();
                return GC_E_CUDA;
            }
            g_dev[dev].grid_hist = sms * (bh < 1 ? 1 : bh);
            g_dev[dev].grid_compact = sms * (bc < 1 ? 1 : bc);
            g_dev[dev].scratch = ptr;
        }
        pd = g_dev[dev];
    }
    unsigned char* sc = static_cast<unsigned char*>(pd.scratch);
    WsView ws;
    ws.hdr = reinterpret_cast<WsHeader*>(sc);
    ws.sel = reinterpret_cast<TensorSel*>(sc + kOffSel);
    ws.hist = reinterpret_cast<uint32_t*>(sc + kOffHist);
    ws.tile_state = reinterpret_cast<unsigned long long*>(sc + kOffState);
    ws.gate = nullptr;
    const TensorDesc* desc = reinterpret_cast<const TensorDesc*>(sc + kOffDesc);
    const uint32_t nt = (n + kTile - 1) / kTile;
    const int gh = (int)(nt < (uint32_t)pd.grid_hist ? nt : (uint32_t)pd.grid_hist);
    const int gcp = (int)(nt < (uint32_t)pd.grid_compact ? nt : (uint32_t)pd.grid_compact);
    k_noalloc_init<<<8, 256, 0, s>>>(sc, n, k, nt);
    k_hist<0, SRC_FOLD><<<gh, kBlock, 0, s>>>(desc, 1u, nt, grad, residual, ws);
    k_hist<1, SRC_RESID><<<gh, kBlock, 0, s>>>(desc, 1u, nt, nullptr, residual, ws);
    k_hist<2, SRC_RESID><<<gh, kBlock, 0, s>>>(desc, 1u, nt, nullptr, residual, ws);
    k_compact<<<gcp, kBlock, 0, s>>>(desc, 1u, nt, residual, out_idx, out_val, nullptr, ws, 0);
    k_noalloc_finish<<<1, 1, 0, s>>>(sc, device_status);
    if (cudaGetLastError() != cudaSuccess) return GC_E_CUDA;
    return GC_OK;
}
