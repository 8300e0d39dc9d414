// Biased model aggregation, Eq. 3:  out[j] = sum_i w_i * x_i[j].
//
// One pass over P + 1 streams: every thread owns one 16-byte column slice at a
// time, issues the P replica loads back to back (P independent 128-bit loads in
// flight per thread), folds them in ascending i with one multiply and P - 1 fused
// multiply-adds, and stores once.  Loads go past L1 (ld.global.cg) with the
// normal L2 policy, stores are marked evict-first.  Evict-first LOADS
// (ld.global.cs) were 11 % slower whenever the L2 still held lines of some other
// buffer written earlier with the normal policy (any real program): such lines
// are never displaced by evict-first traffic, which then has to make do with
// what is left of the L2 (measured: 760 us instead of 687 us for 10 x 109 M
// parameters, in every state but a freshly started process).  The kernel is
// bound by HBM bandwidth: 4 (P + 1) bytes per parameter.
#include "lsgd_internal.cuh"

namespace lsgd {

namespace {

struct AggArgs {
    const float* x[LSGD_MAX_REPLICAS];
    float w[LSGD_MAX_REPLICAS];
};

constexpr int kAggThreads = 256;
constexpr int kAggBatch = 8;  // replica loads kept in flight per thread when P is not a compile-time constant

__device__ __forceinline__ float4 fma4(float w, float4 v, float4 a) {
    a.x = fmaf(w, v.x, a.x);
    a.y = fmaf(w, v.y, a.y);
    a.z = fmaf(w, v.z, a.z);
    a.w = fmaf(w, v.w, a.w);
    return a;
}
__device__ __forceinline__ float4 mul4(float w, float4 v) { return make_float4(w * v.x, w * v.y, w * v.z, w * v.w); }

// PCT > 0: P known at compile time (all loads of a slice in flight at once).
// PCT == 0: any P, replicas taken kAggBatch at a time.
// `out` carries no no-alias promise: it may be one of the replicas (in-place update).
template <int PCT>
__global__ void __launch_bounds__(kAggThreads) aggregate_vec4_kernel(const __grid_constant__ AggArgs a, int P,
                                                                      int64_t n4, int64_t D, float* out) {
    // the up to three elements past the last whole slice: one thread each, same chain of operations
    if (blockIdx.x == 0 && 4 * n4 + threadIdx.x < D) {
        const int64_t j = 4 * n4 + threadIdx.x;
        float acc = a.w[0] * __ldcg(a.x[0] + j);
        for (int r = 1; r < P; ++r) acc = fmaf(a.w[r], __ldcg(a.x[r] + j), acc);
        out[j] = acc;
    }
    const int64_t stride = static_cast<int64_t>(gridDim.x) * kAggThreads;
    for (int64_t i = static_cast<int64_t>(blockIdx.x) * kAggThreads + threadIdx.x; i < n4; i += stride) {
        float4 acc;
        if constexpr (PCT > 0) {
            float4 v[PCT];
#pragma unroll
            for (int r = 0; r < PCT; ++r) v[r] = __ldcg(reinterpret_cast<const float4*>(a.x[r]) + i);
            acc = mul4(a.w[0], v[0]);
#pragma unroll
            for (int r = 1; r < PCT; ++r) acc = fma4(a.w[r], v[r], acc);
        } else {
            acc = make_float4(0.f, 0.f, 0.f, 0.f);
            for (int b = 0; b < P; b += kAggBatch) {
                float4 v[kAggBatch];
#pragma unroll
                for (int u = 0; u < kAggBatch; ++u)
                    if (b + u < P) v[u] = __ldcg(reinterpret_cast<const float4*>(a.x[b + u]) + i);
#pragma unroll
                for (int u = 0; u < kAggBatch; ++u)
                    if (b + u < P) acc = (b + u == 0) ? mul4(a.w[0], v[u]) : fma4(a.w[b + u], v[u], acc);
            }
        }
        __stcs(reinterpret_cast<float4*>(out) + i, acc);
    }
}

// Scalar path: the whole vector when some pointer is not 16-byte aligned (or D < 4).
__global__ void __launch_bounds__(kAggThreads) aggregate_scalar_kernel(const __grid_constant__ AggArgs a, int P,
                                                                        int64_t begin, int64_t D,
                                                                        float* out) {
    const int64_t stride = static_cast<int64_t>(gridDim.x) * kAggThreads;
    for (int64_t j = begin + static_cast<int64_t>(blockIdx.x) * kAggThreads + threadIdx.x; j < D; j += stride) {
        float acc = a.w[0] * __ldcg(a.x[0] + j);
        for (int r = 1; r < P; ++r) acc = fmaf(a.w[r], __ldcg(a.x[r] + j), acc);
        out[j] = acc;
    }
}

template <int PCT>
cudaError_t launch_vec(const AggArgs& a, int P, int64_t n4, int64_t D, float* out, cudaStream_t s) {
    static int blocks_per_sm[64] = {0};
    int dev = 0;
    cudaGetDevice(&dev);
    int& bps = blocks_per_sm[dev & 63];
    if (bps == 0) {
        int b = 0;
        cudaError_t e = cudaOccupancyMaxActiveBlocksPerMultiprocessor(&b, aggregate_vec4_kernel<PCT>, kAggThreads, 0);
        if (e != cudaSuccess) return e;
        bps = b > 0 ? b : 1;
    }
    const int64_t want = (n4 + kAggThreads - 1) / kAggThreads;
    const int64_t cap = static_cast<int64_t>(sm_count()) * bps;
    const int grid = static_cast<int>(want < cap ? want : cap);
    aggregate_vec4_kernel<PCT><<<grid, kAggThreads, 0, s>>>(a, P, n4, D, out);
    return cudaGetLastError();
}

}  // namespace

cudaError_t launch_aggregate(const float* const* replicas, const float* weights, int P, int64_t D, float* out,
                             bool vector_ok, cudaStream_t s) {
    AggArgs a;
    for (int i = 0; i < LSGD_MAX_REPLICAS; ++i) {
        a.x[i] = i < P ? replicas[i] : nullptr;
        a.w[i] = i < P ? weights[i] : 0.f;
    }
    const int64_t n4 = vector_ok ? D / 4 : 0;
    cudaError_t e = cudaSuccess;
    if (n4 > 0) {
        switch (P) {
#define LSGD_AGG_CASE(n) \
    case n:              \
        e = launch_vec<n>(a, P, n4, D, out, s); \
        break;
            LSGD_AGG_CASE(1) LSGD_AGG_CASE(2) LSGD_AGG_CASE(3) LSGD_AGG_CASE(4) LSGD_AGG_CASE(5) LSGD_AGG_CASE(6)
            LSGD_AGG_CASE(7) LSGD_AGG_CASE(8) LSGD_AGG_CASE(9) LSGD_AGG_CASE(10) LSGD_AGG_CASE(11)
            LSGD_AGG_CASE(12) LSGD_AGG_CASE(13) LSGD_AGG_CASE(14) LSGD_AGG_CASE(15) LSGD_AGG_CASE(16)
#undef LSGD_AGG_CASE
            default:
                e = launch_vec<0>(a, P, n4, D, out, s);
        }
        if (e != cudaSuccess) return e;
    }
    const int64_t begin = n4 > 0 ? D : 0;  // the vector kernel takes its own ragged tail along
    if (begin < D) {
        const int64_t rest = D - begin;
        const int64_t want = (rest + kAggThreads - 1) / kAggThreads;
        const int64_t cap = static_cast<int64_t>(sm_count()) * 8;
        aggregate_scalar_kernel<<<static_cast<int>(want < cap ? want : cap), kAggThreads, 0, s>>>(a, P, begin, D, out);
        e = cudaGetLastError();
    }
    return e;
}

}  // namespace lsgd
