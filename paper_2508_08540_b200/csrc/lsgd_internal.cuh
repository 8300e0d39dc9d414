// Internal declarations shared by the translation units of liblsgd.
// Nothing here is part of the C ABI (see include/lsgd.h for that).
#pragma once

#include <cuda_runtime.h>
#include <stdint.h>

#include "lsgd.h"

namespace lsgd {

// ---------------------------------------------------------------------------
// Status block: the first 256 bytes of every scoring / selection workspace.
// Zeroed (together with the selector's histograms) by one clearing kernel per call.
// ---------------------------------------------------------------------------
struct StatusBlock {
    int32_t bad_labels;      // tokens with a label outside [0, C) that is not ignore_index
    int32_t timeout;         // set by a block of the selection kernel whose bounded barrier wait ran out
    uint32_t grid_arrivals;  // the selection kernel's barrier: blocks that have arrived so far, over all its barriers
    uint32_t reserved0;
    unsigned long long stream_ticket;  // dynamic row scheduler of the medium-row scorer
    uint32_t pad[58];
};
static_assert(sizeof(StatusBlock) == 256, "status block is 256 bytes");

constexpr size_t kAlign = 256;
inline size_t align_up(size_t x) { return (x + kAlign - 1) / kAlign * kAlign; }

// ---------------------------------------------------------------------------
// Selector geometry.  Keys are order-preserving 32-bit images of the losses,
// resolved in three radix digits of 11, 11 and 10 bits, most significant first.
// ---------------------------------------------------------------------------
constexpr int kSelPasses = 3;
constexpr int kSelBins = 2048;            // 11-bit digits (the last digit uses 1024 of them)
constexpr int kTile = 4096;               // smallest selection tile (the per-tile counts are sized for it)
constexpr int kSmallN = 1024;             // pools up to this size are sorted by one CTA, one entry per thread
constexpr int kSortBits = 9;              // digits of the stable LSD sort of the selected pairs
constexpr int kSortBins = 1 << kSortBits;
constexpr int kSortMaxRounds = 8;         // a sort tile holds 1024 R entries, R from 1 to 8 (a power of two in the cluster kernels)
constexpr int kSortDirectTiles = 256;     // the launcher grows R before it uses more sort tiles than this
constexpr int kMaxClusterBlocks = 8;      // pools of up to 8 x 8,192 entries run as one cluster (of 16 x 4,096 where the device allows)

struct TopkWorkspace {       // device pointers carved out of the caller's workspace
    StatusBlock* status;
    uint32_t* hist;          // [kSelPasses][kSelBins]
    uint32_t* tile_counts;   // [tiles(N)][4]  (#keys above the threshold, #keys equal to it, largest key, unused)
    uint2* pairs[2];         // [k] ping-pong: (key, index) of the selected entries
    uint32_t* tile_hist;     // [sort tiles][kSortBins] digit counts per sort tile of the current pass
};

// Test hooks (environment, read at every launch): they change launch geometry only, never results.
//   LSGD_TEST_MAX_CTAS=n     no kernel of the scorer or the selector uses more than n thread blocks
//   LSGD_TEST_NO_CLUSTER=1   the selector never runs as a single cluster
//   LSGD_TEST_NARROW_CLUSTER=1  ... and when it does, as 8,192-entry blocks (the variant for devices without 16-block clusters)
// and one that makes the cooperative selector's barrier give up, to test that path without harming the device:
//   LSGD_TEST_PHANTOM_BLOCK=1  the barrier waits for one block more than exist, with a short poll limit (tens of
//                              milliseconds): every block sets the timeout word and returns; outputs are unspecified
struct TestGeometry {
    int max_ctas;      // INT_MAX when unset
    bool no_cluster;
    bool narrow_cluster;
    bool phantom_block;
};
TestGeometry test_geometry();

struct ScoreWorkspace {
    StatusBlock* status;
    float* token_loss;       // [N*T] when T > 1, else unused
};

size_t topk_workspace_bytes(int64_t N, int64_t k);
size_t score_workspace_bytes(int64_t N, int64_t T, int64_t C);
TopkWorkspace carve_topk(void* ws, int64_t N, int64_t k);
ScoreWorkspace carve_score(void* ws, int64_t N, int64_t T, int64_t C);
// Clears the status block and the selector's histograms.  The fused call does this before the scorer runs; a
// selection on its own (launch_topk with `standalone`) clears whatever its kernel needs itself.
cudaError_t zero_topk_workspace(void* ws, int64_t k, cudaStream_t s);

// Launchers (each returns the CUDA error of its launches).  `hist0` non-NULL asks
// the scorer to accumulate the selector's first-digit histogram while it writes
// the losses.
cudaError_t launch_aggregate(const float* const* replicas, const float* weights, int P, int64_t D, float* out,
                             bool vector_ok, cudaStream_t s);
cudaError_t launch_score(const void* logits, lsgd_dtype dt, const int64_t* labels, int64_t N, int64_t T, int64_t C,
                         int64_t ignore_index, float* losses, const ScoreWorkspace& ws, uint32_t* hist0,
                         cudaStream_t s);
cudaError_t launch_topk(const float* losses, int64_t N, int64_t k, lsgd_order order, int32_t* out_idx,
                        float* out_vals, const TopkWorkspace& ws, bool hist0_ready, bool standalone, cudaStream_t s);

int sm_count();  // multiprocessors of the current device (cached per device)

// Launches `kernel` so that it may be scheduled while the previous kernel of the stream is still draining
// (programmatic dependent launch).  Such a kernel must call grid_dependency_wait() before it touches global
// memory: that is where it waits for the previous kernel to have completed, with its writes visible.
template <typename... KArgs, typename... Args>
cudaError_t launch_dependent_smem(void (*kernel)(KArgs...), int grid, int block, size_t smem, cudaStream_t s, Args... args) {
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3(static_cast<unsigned>(grid));
    cfg.blockDim = dim3(static_cast<unsigned>(block));
    cfg.dynamicSmemBytes = smem;
    cfg.stream = s;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr;
    cfg.numAttrs = 1;
    return cudaLaunchKernelEx(&cfg, kernel, static_cast<KArgs>(args)...);
}
template <typename... KArgs, typename... Args>
cudaError_t launch_dependent(void (*kernel)(KArgs...), int grid, int block, cudaStream_t s, Args... args) {
    return launch_dependent_smem(kernel, grid, block, 0, s, args...);
}

// Clears `bytes` (a multiple of 16, 16-byte aligned) of device memory with a kernel that lets the next kernel of the
// stream start at once: a scorer launched with launch_dependent_smem reads its inputs while the head of the workspace
// is still being cleared and waits (grid_dependency_wait) only before it first touches the status block or a histogram.
cudaError_t clear_device_words(void* p, size_t bytes, cudaStream_t s);

// ---------------------------------------------------------------------------
// Device helpers
// ---------------------------------------------------------------------------
#ifdef __CUDACC__

// Programmatic dependent launch, device side.  grid_launch_dependents: the next kernel of the stream may start
// being scheduled once every CTA of this grid has got here (or exited).  grid_dependency_wait: blocks until the
// previous kernel has completed and its memory is visible; a no-op for a normally launched kernel.
__device__ __forceinline__ void grid_launch_dependents() { asm volatile("griddepcontrol.launch_dependents;" ::: "memory"); }
__device__ __forceinline__ void grid_dependency_wait() { asm volatile("griddepcontrol.wait;" ::: "memory"); }

// Order-preserving key of a loss: larger key = selected earlier.  -0 maps to +0,
// every NaN maps to the largest key (it ranks above +inf).
__device__ __forceinline__ uint32_t loss_key(float v) {
    uint32_t u = __float_as_uint(v);
    if (v != v) return 0xFFFFFFFFu;
    if (u == 0x80000000u) u = 0u;
    return (u & 0x80000000u) ? ~u : (u | 0x80000000u);
}

__device__ __forceinline__ float warp_max(float v) {
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) v = fmaxf(v, __shfl_xor_sync(0xFFFFFFFFu, v, o));
    return v;
}
__device__ __forceinline__ float warp_sum(float v) {
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xFFFFFFFFu, v, o);
    return v;
}
__device__ __forceinline__ int warp_sum(int v) {
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xFFFFFFFFu, v, o);
    return v;
}

#endif  // __CUDACC__

}  // namespace lsgd
