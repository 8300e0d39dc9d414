// lsgd_topk_select_static: the selector of lsgd_topk_select for callers that
// cannot hand the library a workspace because they cannot allocate one.
//
// Some code that wants the top-k runs where device allocation is off the table:
// inside a region that must not call cudaMalloc (a latency-critical loop, a
// callback on a stream, a process whose memory pool is owned by another
// framework and fully handed out), or in a host program that simply has no
// allocator for device memory wired in.  For them the scratch space lives in
// this library's own image: a fixed array in device global memory that every
// GPU which loads the library carries until the process exits.
#include <atomic>
#include <mutex>

#include "lsgd_internal.cuh"

namespace lsgd {
namespace {

// Workspace of the selector at N = k = LSGD_STATIC_TOPK_MAX_N, spelled out so
// that it is a compile-time constant (checked against the run-time formula below).
constexpr size_t kMaxN = LSGD_STATIC_TOPK_MAX_N;
constexpr size_t kMaxTiles = (kMaxN + kTile - 1) / kTile;
constexpr size_t kMaxSortTiles = kSortDirectTiles;  // pools of this size never use more sort tiles
static_assert(kMaxN <= size_t{kSortDirectTiles} * 1024 * kSortMaxRounds, "the sort's tile bound covers the largest pool");
constexpr size_t up256(size_t x) { return (x + 255) / 256 * 256; }
constexpr size_t kScratchBytes = sizeof(StatusBlock) + up256(sizeof(uint32_t) * kSelPasses * kSelBins) +
                                 up256(sizeof(uint32_t) * kMaxSortTiles * kSortBins) +
                                 up256(sizeof(uint32_t) * 4 * kMaxTiles) + 4 * up256(sizeof(uint32_t) * kMaxN);

// The scratch itself.  In host code this name is only a handle for the runtime's
// symbol table, never an address a kernel may be given: the device address is
// asked for once per device with cudaGetSymbolAddress.
static __device__ __align__(256) unsigned char g_static_topk_scratch[kScratchBytes];

constexpr int kMaxDevices = 64;
std::mutex g_setup_mutex;
std::atomic<void*> g_scratch_addr[kMaxDevices];

// Device address of the scratch array on the current device (looked up on the
// first call per device, with that device current), or nullptr on failure.
void* scratch_on_current_device() {
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= kMaxDevices) return nullptr;
    void* p = g_scratch_addr[dev].load(std::memory_order_acquire);
    if (p) return p;
    std::lock_guard<std::mutex> lock(g_setup_mutex);
    p = g_scratch_addr[dev].load(std::memory_order_acquire);
    if (p) return p;
    void* addr = nullptr;
    if (cudaGetSymbolAddress(&addr, g_static_topk_scratch) != cudaSuccess || !addr) return nullptr;
    g_scratch_addr[dev].store(addr, std::memory_order_release);
    return addr;
}

bool aligned4(const void* p) { return (reinterpret_cast<uintptr_t>(p) & 3) == 0; }

}  // namespace
}  // namespace lsgd

using namespace lsgd;

extern "C" lsgd_status lsgd_topk_select_static(const float* losses, int64_t N, int64_t k, lsgd_order order,
                                               int32_t* out_idx, float* out_vals, void* cuda_stream) {
    if (order != LSGD_ORDER_LOSS_DESC && order != LSGD_ORDER_INDEX_ASC) return LSGD_ERR_UNSUPPORTED;
    if (N < 0 || k < 0 || k > N) return LSGD_ERR_INVALID_ARG;
    if (N > static_cast<int64_t>(kMaxN)) return LSGD_ERR_UNSUPPORTED;  // beyond the built-in scratch
    if (k == 0) return LSGD_OK;
    if (!losses || !out_idx) return LSGD_ERR_INVALID_ARG;
    if (!aligned4(losses) || !aligned4(out_idx) || (out_vals && !aligned4(out_vals))) return LSGD_ERR_ALIGNMENT;
    if (topk_workspace_bytes(N, k) > kScratchBytes) return LSGD_ERR_WORKSPACE;  // cannot happen for N <= kMaxN
    void* ws = scratch_on_current_device();
    if (!ws) return LSGD_ERR_CUDA;
    cudaStream_t s = static_cast<cudaStream_t>(cuda_stream);
    // the array keeps whatever the previous call left: the launcher clears what its kernel needs to start at zero
    // (the status block and the digit histograms)
    return launch_topk(losses, N, k, order, out_idx, out_vals, carve_topk(ws, N, k), false, true, s) == cudaSuccess
               ? LSGD_OK
               : LSGD_ERR_CUDA;
}
