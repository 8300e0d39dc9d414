// One round's aggregation as the training loop uses it (Eq. 3; Section 2's update
// rule; Algorithm 1: after the aggregation every worker continues from x_{t+1}).
//
//   x_{t+1}[j] = sum_i w_i x_i[j]                        (Eq. 3), or
//   x_{t+1}[j] = b[j] + sum_i w_i (x_i[j] - b[j])        (the same update written around b = x_t)
//
// over fp32 or bf16 replicas with fp32 accumulation in ascending i, written to
// an fp32 vector and, on request, back into all P replicas in the same pass, so
// that the next local phase starts without a second sweep over the model.
//
// Same shape as the plain Eq. 3 kernel: a thread owns one 16-byte slice of every
// replica (4 fp32 or 8 bf16 parameters), keeps up to kBatch replica loads in
// flight, folds them in order, stores once per destination.  HBM-bound:
//   P e (+ 4) bytes read and (4 +) P e written per parameter, e = bytes per replica element.
#include <cuda_bf16.h>

#include "lsgd_internal.cuh"

namespace lsgd {
namespace {

struct RoundArgs {
    void* x[LSGD_MAX_REPLICAS];
    float w[LSGD_MAX_REPLICAS];
};

constexpr int kThreads = 256;
constexpr int kBatch = 16;  // replica loads (16 bytes each, kept raw until they are folded) in flight per thread

template <typename T>
struct Slice;  // how the 16-byte slice of a replica that one thread handles maps to parameters

template <>
struct Slice<float> {
    static constexpr int kElems = 4;
    __device__ __forceinline__ static void widen(const uint4& q, float (&v)[4]) {
        v[0] = __uint_as_float(q.x); v[1] = __uint_as_float(q.y); v[2] = __uint_as_float(q.z); v[3] = __uint_as_float(q.w);
    }
    __device__ __forceinline__ static void store(void* p, int64_t i, const float (&r)[4]) {
        __stcs(reinterpret_cast<float4*>(p) + i, make_float4(r[0], r[1], r[2], r[3]));
    }
    __device__ __forceinline__ static float load_one(const void* p, int64_t j) { return __ldcg(static_cast<const float*>(p) + j); }
    __device__ __forceinline__ static void store_one(void* p, int64_t j, float r) { static_cast<float*>(p)[j] = r; }
};

template <>
struct Slice<__nv_bfloat16> {
    static constexpr int kElems = 8;
    __device__ __forceinline__ static void widen(const uint4& q, float (&v)[8]) {
        const uint32_t u[4] = {q.x, q.y, q.z, q.w};
#pragma unroll
        for (int h = 0; h < 4; ++h) {  // bf16 is the upper half of an fp32: widening is exact
            v[2 * h] = __uint_as_float(u[h] << 16);
            v[2 * h + 1] = __uint_as_float(u[h] & 0xFFFF0000u);
        }
    }
    __device__ __forceinline__ static uint32_t pack(float lo, float hi) {
        const __nv_bfloat162 b = __floats2bfloat162_rn(lo, hi);  // round to nearest even
        return *reinterpret_cast<const uint32_t*>(&b);
    }
    __device__ __forceinline__ static void store(void* p, int64_t i, const float (&r)[8]) {
        __stcs(reinterpret_cast<uint4*>(p) + i,
               make_uint4(pack(r[0], r[1]), pack(r[2], r[3]), pack(r[4], r[5]), pack(r[6], r[7])));
    }
    __device__ __forceinline__ static float load_one(const void* p, int64_t j) {
        return __uint_as_float(static_cast<uint32_t>(static_cast<const uint16_t*>(p)[j]) << 16);
    }
    __device__ __forceinline__ static void store_one(void* p, int64_t j, float r) {
        static_cast<__nv_bfloat16*>(p)[j] = __float2bfloat16_rn(r);
    }
};

// Vector path over slices [0, n_slices).  BASE: delta form around `base`.  BCAST: write x_{t+1} into every replica.
template <typename T, bool BASE, bool BCAST>
__global__ void __launch_bounds__(kThreads, 2)
aggregate_round_kernel(const __grid_constant__ RoundArgs a, int P, int64_t n_slices, const float* base, float* out) {
    constexpr int E = Slice<T>::kElems;
    const int64_t stride = static_cast<int64_t>(gridDim.x) * kThreads;
    for (int64_t i = static_cast<int64_t>(blockIdx.x) * kThreads + threadIdx.x; i < n_slices; i += stride) {
        float b[E], acc[E];
        if (BASE) {
#pragma unroll
            for (int q = 0; q < E / 4; ++q) {
                const float4 t = __ldcg(reinterpret_cast<const float4*>(base) + i * (E / 4) + q);
                b[4 * q] = t.x; b[4 * q + 1] = t.y; b[4 * q + 2] = t.z; b[4 * q + 3] = t.w;
            }
        }
        for (int r0 = 0; r0 < P; r0 += kBatch) {
            uint4 raw[kBatch];
#pragma unroll
            for (int u = 0; u < kBatch; ++u)
                if (r0 + u < P) raw[u] = __ldcg(reinterpret_cast<const uint4*>(a.x[r0 + u]) + i);
#pragma unroll
            for (int u = 0; u < kBatch; ++u)
                if (r0 + u < P) {
                    const float w = a.w[r0 + u];
                    float v[E];
                    Slice<T>::widen(raw[u], v);
#pragma unroll
                    for (int e = 0; e < E; ++e) {
                        const float d = BASE ? v[e] - b[e] : v[e];
                        acc[e] = (r0 + u == 0) ? w * d : fmaf(w, d, acc[e]);
                    }
                }
        }
        if (BASE) {
#pragma unroll
            for (int e = 0; e < E; ++e) acc[e] += b[e];
        }
        if (out) {
#pragma unroll
            for (int q = 0; q < E / 4; ++q)
                __stcs(reinterpret_cast<float4*>(out) + i * (E / 4) + q,
                       make_float4(acc[4 * q], acc[4 * q + 1], acc[4 * q + 2], acc[4 * q + 3]));
        }
        if (BCAST) {
            for (int r = 0; r < P; ++r) Slice<T>::store(a.x[r], i, acc);
        }
    }
}

// Element path: the ragged tail [begin, D) of the vector path, or everything when a pointer is not 16-byte aligned.
template <typename T, bool BASE, bool BCAST>
__global__ void __launch_bounds__(kThreads)
aggregate_round_scalar_kernel(const __grid_constant__ RoundArgs a, int P, int64_t begin, int64_t D, const float* base,
                              float* out) {
    const int64_t stride = static_cast<int64_t>(gridDim.x) * kThreads;
    for (int64_t j = begin + static_cast<int64_t>(blockIdx.x) * kThreads + threadIdx.x; j < D; j += stride) {
        const float b = BASE ? base[j] : 0.f;
        float acc = 0.f;
        for (int r = 0; r < P; ++r) {
            const float v = Slice<T>::load_one(a.x[r], j);
            const float d = BASE ? v - b : v;
            acc = r == 0 ? a.w[0] * d : fmaf(a.w[r], d, acc);
        }
        if (BASE) acc += b;
        if (out) out[j] = acc;
        if (BCAST)
            for (int r = 0; r < P; ++r) Slice<T>::store_one(a.x[r], j, acc);
    }
}

template <typename T, bool BASE, bool BCAST>
cudaError_t launch_variant(const RoundArgs& a, int P, int64_t D, const float* base, float* out, bool vector_ok,
                           cudaStream_t s) {
    constexpr int E = Slice<T>::kElems;
    const int64_t n_slices = vector_ok ? D / E : 0;
    if (n_slices > 0) {
        static int blocks_per_sm[64] = {0};
        int dev = 0;
        cudaGetDevice(&dev);
        int& bps = blocks_per_sm[dev & 63];
        if (bps == 0) {
            int n = 0;
            const cudaError_t e = cudaOccupancyMaxActiveBlocksPerMultiprocessor(
                &n, aggregate_round_kernel<T, BASE, BCAST>, kThreads, 0);
            if (e != cudaSuccess) return e;
            bps = n > 0 ? n : 1;
        }
        const int64_t want = (n_slices + kThreads - 1) / kThreads;
        const int64_t cap = static_cast<int64_t>(sm_count()) * bps;
        aggregate_round_kernel<T, BASE, BCAST><<<static_cast<int>(want < cap ? want : cap), kThreads, 0, s>>>(
            a, P, n_slices, base, out);
        const cudaError_t e = cudaGetLastError();
        if (e != cudaSuccess) return e;
    }
    const int64_t begin = n_slices * E;
    if (begin < D) {
        const int64_t want = (D - begin + kThreads - 1) / kThreads;
        const int64_t cap = static_cast<int64_t>(sm_count()) * 8;
        aggregate_round_scalar_kernel<T, BASE, BCAST><<<static_cast<int>(want < cap ? want : cap), kThreads, 0, s>>>(
            a, P, begin, D, base, out);
    }
    return cudaGetLastError();
}

template <typename T>
cudaError_t launch_dtype(const RoundArgs& a, int P, int64_t D, const float* base, float* out, bool bcast, bool vec,
                         cudaStream_t s) {
    if (base) return bcast ? launch_variant<T, true, true>(a, P, D, base, out, vec, s)
                           : launch_variant<T, true, false>(a, P, D, base, out, vec, s);
    return bcast ? launch_variant<T, false, true>(a, P, D, base, out, vec, s)
                 : launch_variant<T, false, false>(a, P, D, base, out, vec, s);
}

bool aligned_to(const void* p, size_t a) { return (reinterpret_cast<uintptr_t>(p) & (a - 1)) == 0; }

// 0: disjoint, 1: the same range, 2: partial overlap
int relation(const void* a, size_t na, const void* b, size_t nb) {
    const uintptr_t a0 = reinterpret_cast<uintptr_t>(a), b0 = reinterpret_cast<uintptr_t>(b);
    if (a0 == b0 && na == nb) return 1;
    return (a0 < b0 + nb && b0 < a0 + na) ? 2 : 0;
}

}  // namespace
}  // namespace lsgd

using namespace lsgd;

extern "C" lsgd_status lsgd_aggregate_round(void* const* replicas, lsgd_dtype dtype, const float* weights, int32_t P,
                                            int64_t D, const float* base, float* out, int32_t broadcast,
                                            void* cuda_stream) {
    if (dtype != LSGD_F32 && dtype != LSGD_BF16) return LSGD_ERR_UNSUPPORTED;
    if (P < 1 || P > LSGD_MAX_REPLICAS || D < 0 || !replicas || !weights) return LSGD_ERR_INVALID_ARG;
    if (!out && !broadcast) return LSGD_ERR_INVALID_ARG;  // the result would go nowhere
    if (D == 0) return LSGD_OK;
    const size_t es = dtype == LSGD_F32 ? 4 : 2;
    const size_t rep_bytes = es * static_cast<size_t>(D), f32_bytes = 4 * static_cast<size_t>(D);
    bool vec = (!out || aligned_to(out, 16)) && (!base || aligned_to(base, 16));
    if ((out && !aligned_to(out, 4)) || (base && !aligned_to(base, 4))) return LSGD_ERR_ALIGNMENT;
    RoundArgs a;
    for (int i = 0; i < LSGD_MAX_REPLICAS; ++i) {
        a.x[i] = i < P ? replicas[i] : nullptr;
        a.w[i] = i < P ? weights[i] : 0.f;
    }
    for (int i = 0; i < P; ++i) {
        if (!replicas[i]) return LSGD_ERR_INVALID_ARG;
        if (!aligned_to(replicas[i], es)) return LSGD_ERR_ALIGNMENT;
        vec = vec && aligned_to(replicas[i], 16);
        // a thread reads its slice of every source before it writes that slice anywhere, so exact aliases are safe
        // wherever the element sizes agree; partial overlaps are not
        if (out) {
            const int r = relation(replicas[i], rep_bytes, out, f32_bytes);
            if (r == 2 || (r == 1 && dtype != LSGD_F32)) return LSGD_ERR_INVALID_ARG;
        }
        if (base) {
            const int r = relation(replicas[i], rep_bytes, base, f32_bytes);
            if (r == 2 || (r == 1 && dtype != LSGD_F32)) return LSGD_ERR_INVALID_ARG;
        }
        if (broadcast)
            for (int j = 0; j < i; ++j)
                if (relation(replicas[i], rep_bytes, replicas[j], rep_bytes) != 0) return LSGD_ERR_INVALID_ARG;
    }
    if (out && base && relation(out, f32_bytes, base, f32_bytes) == 2) return LSGD_ERR_INVALID_ARG;
    cudaStream_t s = static_cast<cudaStream_t>(cuda_stream);
    const cudaError_t e = dtype == LSGD_F32
                              ? launch_dtype<float>(a, P, D, base, out, broadcast != 0, vec, s)
                              : launch_dtype<__nv_bfloat16>(a, P, D, base, out, broadcast != 0, vec, s);
    return e == cudaSuccess ? LSGD_OK : LSGD_ERR_CUDA;
}
