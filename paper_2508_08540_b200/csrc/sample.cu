// Per-epoch data allocation (Section 4.2; Algorithm 1, the steps before the
// training loop): how many samples each worker group gets, the uniform draws
// without replacement, and the fast workers' allocation (highest-loss samples
// first, the remainder drawn from the unselected samples).
//
// A draw gives every sample an independent random priority and keeps the
// candidates with the highest priorities, ties by lower index.  That is the same
// total order as the loss-based selection, so the draw runs on the selector:
// a kernel writes the priorities as a table the selector can read (30-bit
// integers stored as the bit patterns of non-negative finite floats, whose order
// as floats is their order as integers), excluded samples are set to -inf,
// which ranks below every priority, and the selector returns the first n_draw
// entries in priority order.  No arithmetic is ever done on the table's values.
//
// Priorities come from Philox4x32 with 10 rounds (Salmon, Moraes, Dror, Shaw,
// SC'11), a counter-based generator: the value of sample i depends only on
// (seed, stream, i), so results do not depend on the launch geometry.
#include <algorithm>
#include <cmath>

#include "lsgd_internal.cuh"

namespace lsgd {
namespace {

constexpr int kThreads = 256;

struct Philox4 {
    uint32_t w[4];
};

// One Philox4x32-10 block.  Round: (c0, c1, c2, c3) <- (hi(M1 c2) ^ c1 ^ k0, lo(M1 c2), hi(M0 c0) ^ c3 ^ k1, lo(M0 c0));
// the key advances by the two Weyl constants after every round.
__device__ __forceinline__ Philox4 philox4x32_10(uint32_t c0, uint32_t c1, uint32_t c2, uint32_t c3, uint32_t k0,
                                                 uint32_t k1) {
    constexpr uint32_t kM0 = 0xD2511F53u, kM1 = 0xCD9E8D57u, kW0 = 0x9E3779B9u, kW1 = 0xBB67AE85u;
#pragma unroll
    for (int r = 0; r < 10; ++r) {
        const uint32_t hi0 = __umulhi(kM0, c0), lo0 = kM0 * c0;
        const uint32_t hi1 = __umulhi(kM1, c2), lo1 = kM1 * c2;
        c0 = hi1 ^ c1 ^ k0;
        c1 = lo1;
        c2 = hi0 ^ c3 ^ k1;
        c3 = lo0;
        k0 += kW0;
        k1 += kW1;
    }
    return Philox4{{c0, c1, c2, c3}};
}

// pri[i] = bit pattern (word (i mod 4) of block (i div 4)) >> 2, for i < N.  One thread per block of four samples;
// `pri` is 16-byte aligned (it lives in the workspace), so full blocks are stored as one vector.
__global__ void __launch_bounds__(kThreads)
priority_kernel(float* __restrict__ pri, int64_t N, uint32_t seed_lo, uint32_t seed_hi, uint32_t stream_lo,
                uint32_t stream_hi) {
    const int64_t blocks = (N + 3) >> 2;
    for (int64_t b = static_cast<int64_t>(blockIdx.x) * kThreads + threadIdx.x; b < blocks;
         b += static_cast<int64_t>(gridDim.x) * kThreads) {
        const Philox4 p = philox4x32_10(static_cast<uint32_t>(b), 0u, stream_lo, stream_hi, seed_lo, seed_hi);
        const float4 v = make_float4(__uint_as_float(p.w[0] >> 2), __uint_as_float(p.w[1] >> 2),
                                     __uint_as_float(p.w[2] >> 2), __uint_as_float(p.w[3] >> 2));
        const int64_t i = b << 2;
        if (i + 4 <= N) {
            reinterpret_cast<float4*>(pri)[b] = v;
        } else {
            pri[i] = v.x;
            if (i + 1 < N) pri[i + 1] = v.y;
            if (i + 2 < N) pri[i + 2] = v.z;
        }
    }
}

// Takes the listed samples out of the draw.  Entries outside [0, N) are ignored.
__global__ void __launch_bounds__(kThreads)
exclude_kernel(float* __restrict__ pri, int64_t N, const int32_t* __restrict__ exclude_idx, int64_t n_exclude) {
    for (int64_t j = static_cast<int64_t>(blockIdx.x) * kThreads + threadIdx.x; j < n_exclude;
         j += static_cast<int64_t>(gridDim.x) * kThreads) {
        const int32_t e = exclude_idx[j];
        if (e >= 0 && e < N) pri[e] = __uint_as_float(0xFF800000u);  // -inf
    }
}

int grid_for(int64_t items) {
    const int64_t ctas = (items + kThreads - 1) / kThreads;
    return static_cast<int>(std::max<int64_t>(1, std::min<int64_t>(ctas, static_cast<int64_t>(sm_count()) * 8)));
}

bool aligned_to(const void* p, size_t a) { return (reinterpret_cast<uintptr_t>(p) & (a - 1)) == 0; }

// Workspace of a draw of at most `m` out of N: the selector's workspace for (N, m), then the priority table.
size_t draw_ws_bytes(int64_t N, int64_t m) { return topk_workspace_bytes(N, m) + align_up(sizeof(float) * static_cast<size_t>(N)); }

lsgd_status check_ws(const void* ws, size_t have, size_t need) {
    if (!ws) return LSGD_ERR_INVALID_ARG;
    if (!aligned_to(ws, kAlign)) return LSGD_ERR_ALIGNMENT;
    if (have < need) return LSGD_ERR_WORKSPACE;
    return LSGD_OK;
}

// Enqueues one draw.  `sel_bytes` is where the priority table starts inside the workspace.
cudaError_t enqueue_draw(int64_t N, int64_t m, uint64_t seed, uint64_t stream, const int32_t* exclude_idx,
                         int64_t n_exclude, int32_t* out_idx, void* ws, size_t sel_bytes, cudaStream_t s) {
    float* pri = reinterpret_cast<float*>(static_cast<unsigned char*>(ws) + sel_bytes);
    cudaError_t e = cudaSuccess;
    priority_kernel<<<grid_for((N + 3) / 4), kThreads, 0, s>>>(pri, N, static_cast<uint32_t>(seed),
                                                               static_cast<uint32_t>(seed >> 32),
                                                               static_cast<uint32_t>(stream),
                                                               static_cast<uint32_t>(stream >> 32));
    if (n_exclude > 0) exclude_kernel<<<grid_for(n_exclude), kThreads, 0, s>>>(pri, N, exclude_idx, n_exclude);
    e = cudaGetLastError();
    if (e != cudaSuccess) return e;
    return launch_topk(pri, N, m, LSGD_ORDER_LOSS_DESC, out_idx, nullptr, carve_topk(ws, N, m), false, true, s);
}

}  // namespace
}  // namespace lsgd

using namespace lsgd;

extern "C" {

lsgd_status lsgd_allocation_sizes(int64_t N, int32_t tau_fast, int32_t p_fast, int32_t tau_slow, int32_t p_slow,
                                  double lambda, int64_t* n_fast, int64_t* n_slow, int64_t* k_high) {
    if (!n_fast || !n_slow || !k_high) return LSGD_ERR_INVALID_ARG;
    if (N < 0 || tau_fast < 0 || p_fast < 0 || tau_slow < 0 || p_slow < 0) return LSGD_ERR_INVALID_ARG;
    if (!(lambda >= 0.0 && lambda <= 1.0)) return LSGD_ERR_INVALID_ARG;
    const unsigned __int128 a = static_cast<unsigned __int128>(tau_fast) * static_cast<uint32_t>(p_fast);
    const unsigned __int128 b = static_cast<unsigned __int128>(tau_slow) * static_cast<uint32_t>(p_slow);
    if (a + b == 0) return LSGD_ERR_INVALID_ARG;
    const int64_t nf = static_cast<int64_t>(a * static_cast<unsigned __int128>(N) / (a + b));
    // floor(lambda N_F); a product that misses the next integer by no more than the rounding of a decimal lambda
    // and of the multiplication (2^-51 relative) is that integer: 0.29 * 100 = 28.999999999999996 gives 29
    const double prod = lambda * static_cast<double>(nf);
    double kf = std::floor(prod);
    if ((kf + 1.0) - prod <= (kf + 1.0) * 0x1p-51) kf += 1.0;
    const int64_t k = static_cast<int64_t>(kf);
    *n_fast = nf;
    *n_slow = N - nf;
    *k_high = std::min(std::max<int64_t>(k, 0), nf);
    return LSGD_OK;
}

lsgd_status lsgd_worker_share(int64_t n, int32_t P, int32_t p, int64_t* begin, int64_t* end) {
    if (!begin || !end || n < 0 || P < 1 || p < 0 || p >= P) return LSGD_ERR_INVALID_ARG;
    *begin = static_cast<int64_t>(static_cast<unsigned __int128>(n) * static_cast<uint32_t>(p) / static_cast<uint32_t>(P));
    *end = static_cast<int64_t>(static_cast<unsigned __int128>(n) * (static_cast<uint32_t>(p) + 1u) / static_cast<uint32_t>(P));
    return LSGD_OK;
}

size_t lsgd_draw_workspace_bytes(int64_t N, int64_t n_draw) {
    if (N < 0 || n_draw < 0 || n_draw > N) return 0;
    return draw_ws_bytes(N, n_draw);
}

lsgd_status lsgd_draw_uniform(int64_t N, int64_t n_draw, uint64_t seed, uint64_t stream, const int32_t* exclude_idx,
                              int64_t n_exclude, int32_t* out_idx, void* ws, size_t ws_bytes, void* cuda_stream) {
    if (N < 0 || n_draw < 0 || n_exclude < 0 || n_exclude > N || n_draw > N - n_exclude) return LSGD_ERR_INVALID_ARG;
    if (N >= (int64_t{1} << 31)) return LSGD_ERR_UNSUPPORTED;
    if (n_draw == 0) return LSGD_OK;
    if (!out_idx || (n_exclude > 0 && !exclude_idx)) return LSGD_ERR_INVALID_ARG;
    if (!aligned_to(out_idx, 4) || !aligned_to(exclude_idx, 4)) return LSGD_ERR_ALIGNMENT;
    const lsgd_status st = check_ws(ws, ws_bytes, draw_ws_bytes(N, n_draw));
    if (st != LSGD_OK) return st;
    const cudaError_t e = enqueue_draw(N, n_draw, seed, stream, exclude_idx, n_exclude, out_idx, ws,
                                       topk_workspace_bytes(N, n_draw), static_cast<cudaStream_t>(cuda_stream));
    return e == cudaSuccess ? LSGD_OK : LSGD_ERR_CUDA;
}

size_t lsgd_fast_allocation_workspace_bytes(int64_t N, int64_t k_high, int64_t n_fill) {
    if (N < 0 || k_high < 0 || n_fill < 0 || k_high > N || n_fill > N - k_high) return 0;
    return draw_ws_bytes(N, std::max(k_high, n_fill));
}

lsgd_status lsgd_fast_allocation(const float* losses, int64_t N, int64_t k_high, int64_t n_fill, uint64_t seed,
                                 uint64_t stream, int32_t* out_idx, void* ws, size_t ws_bytes, void* cuda_stream) {
    if (N < 0 || k_high < 0 || n_fill < 0 || k_high > N || n_fill > N - k_high) return LSGD_ERR_INVALID_ARG;
    if (N >= (int64_t{1} << 31)) return LSGD_ERR_UNSUPPORTED;
    if (k_high + n_fill == 0) return LSGD_OK;
    if (!out_idx || (k_high > 0 && !losses)) return LSGD_ERR_INVALID_ARG;
    if (!aligned_to(out_idx, 4) || !aligned_to(losses, 4)) return LSGD_ERR_ALIGNMENT;
    const int64_t kmax = std::max(k_high, n_fill);
    const lsgd_status st = check_ws(ws, ws_bytes, draw_ws_bytes(N, kmax));
    if (st != LSGD_OK) return st;
    cudaStream_t s = static_cast<cudaStream_t>(cuda_stream);
    if (k_high > 0) {
        if (launch_topk(losses, N, k_high, LSGD_ORDER_LOSS_DESC, out_idx, nullptr, carve_topk(ws, N, k_high), false, true, s) !=
            cudaSuccess)
            return LSGD_ERR_CUDA;
    }
    if (n_fill > 0) {
        // the same workspace, re-carved for the draw: the stream orders it after the selection above
        if (enqueue_draw(N, n_fill, seed, stream, out_idx, k_high, out_idx + k_high, ws, topk_workspace_bytes(N, kmax),
                         s) != cudaSuccess)
            return LSGD_ERR_CUDA;
    }
    return LSGD_OK;
}

}  // extern "C"
