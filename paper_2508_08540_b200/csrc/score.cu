// Per-sample loss record (Algorithm 1: "record all individual loss of processed
// data"): softmax cross-entropy per row of the candidate pool, mean over the
// unmasked tokens of a sample.
//
// Every row is evaluated as
//     m  = max_j x_j
//     s' = sum over all j except ONE occurrence of the maximum of exp(x_j - m)
//     l  = (m - x_y) + log1p(s')
// which is the textbook  (m - x_y) + log(sum_j exp(x_j - m))  with the term that
// equals exactly 1 taken out of the sum, so that losses near zero keep their
// relative accuracy in fp32.  exp(x_j - m) is evaluated as
//     ex2(fma(x_j, L, -fl(m L)))      with L = fl(log2 e),
// whose argument equals (x_j - m) L + d with d = fma(m, L, -fl(m L)) known
// exactly; the common factor 2^d is divided out once per row.
//
// Three row shapes, three kernels (all bound by the bytes of the logits):
//   tiny rows   (C <= 32)         one thread per row out of a shared-memory tile
//   short rows  (<= 4064 bytes)   one warp per row, the row held in registers
//   long rows   (<= ~200 KB)      one CTA per row, the row brought into shared
//                                 memory by bulk asynchronous copies (TMA, 1-D)
//   anything longer               one CTA per row, two passes over global memory
// Rows whose label is ignore_index are never read.
#include <cuda_bf16.h>

#include <algorithm>

#include "lsgd_internal.cuh"

namespace lsgd {

namespace {

constexpr float kLog2e = 1.4426950408889634f;
constexpr uint32_t kWaitLimit = 1u << 20;  // polls (of up to ~2 us each) of a bulk-copy barrier before giving up

__device__ __forceinline__ float ex2(float x) {
    float y;
    asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
    return y;
}
__device__ __forceinline__ float neg_inf() { return __uint_as_float(0xFF800000u); }

template <typename T>
struct Elem;
template <>
struct Elem<float> {
    static constexpr int kPerVec = 4;
    __device__ static float widen(float v) { return v; }
    __device__ static float neg_inf_elem() { return neg_inf(); }
};
template <>
struct Elem<__nv_bfloat16> {
    static constexpr int kPerVec = 8;
    __device__ static float widen(__nv_bfloat16 v) { return __bfloat162float(v); }
    __device__ static __nv_bfloat16 neg_inf_elem() { return __ushort_as_bfloat16(0xFF80u); }
};

// Row constants for the exponentials:  ex2(fma(x, L, nml)) = 2^d * exp(x - m).
struct RowScale {
    float nml;   // -fl(m L)
    float corr;  // 2^-d
    __device__ explicit RowScale(float m) {
        const float p = m * kLog2e;
        nml = -p;
        corr = ex2(-fmaf(m, kLog2e, -p));
    }
};

// Final formula.  s_lt: sum of 2^d exp(x_j - m) over the x_j below the maximum;
// n_max: how many x_j equal the maximum.
__device__ __forceinline__ float finish_loss(float m, float xy, float s_lt, int n_max, const RowScale& rs) {
    const float s_excl = fmaf(s_lt, rs.corr, static_cast<float>(n_max - 1));
    return (m - xy) + log1pf(s_excl);
}

// The selector's first radix digit, accumulated per CTA in shared memory.
struct Hist0 {
    uint32_t* smem;
    uint32_t* global;
    __device__ void clear() {
        if (global)
            for (int i = threadIdx.x; i < kSelBins; i += blockDim.x) smem[i] = 0;
    }
    __device__ void add(float loss) {
        if (global) atomicAdd(&smem[loss_key(loss) >> 21], 1u);
    }
    __device__ void flush() {
        if (global)
            for (int i = threadIdx.x; i < kSelBins; i += blockDim.x)
                if (smem[i]) atomicAdd(&global[i], smem[i]);
    }
};

// label checks shared by all kernels: returns 0 = score it, 1 = ignored, 2 = bad
__device__ __forceinline__ int label_class(int64_t y, int64_t C, int64_t ignore_index) {
    if (y == ignore_index) return 1;
    return (y < 0 || y >= C) ? 2 : 0;
}

// ---------------------------------------------------------------------------
// Tiny rows: a CTA stages 256 consecutive rows (contiguous in memory) into
// shared memory with coalesced element loads; each thread then owns one row.
// ---------------------------------------------------------------------------
constexpr int kTinyThreads = 256;
constexpr int kTinyMaxC = 32;

template <typename T>
__global__ void __launch_bounds__(kTinyThreads)
score_tiny_rows_kernel(const T* __restrict__ logits, const int64_t* __restrict__ labels, int64_t rows, int C,
                       int64_t ignore_index, float* __restrict__ row_loss, StatusBlock* status, uint32_t* hist0) {
    __shared__ float tile[kTinyThreads * (kTinyMaxC + 1)];
    __shared__ uint32_t hist_s[kSelBins];
    Hist0 h{hist_s, hist0};
    h.clear();
    const int pitch = C | 1;  // odd pitch: conflict-free row reads
    const int64_t tiles = (rows + kTinyThreads - 1) / kTinyThreads;
    for (int64_t t = blockIdx.x; t < tiles; t += gridDim.x) {
        const int64_t row0 = t * kTinyThreads;
        const int nrows = rows - row0 < kTinyThreads ? static_cast<int>(rows - row0) : kTinyThreads;
        const T* src = logits + row0 * C;
        const int n = nrows * C;
        __syncthreads();
        for (int i = threadIdx.x; i < n; i += kTinyThreads) {
            const int r = i / C;
            tile[r * pitch + (i - r * C)] = Elem<T>::widen(src[i]);
        }
        __syncthreads();
        if (threadIdx.x < nrows) {
            const int64_t row = row0 + threadIdx.x;
            const int64_t y = labels[row];
            const int cls = label_class(y, C, ignore_index);
            float loss = 0.f;
            if (cls == 2) {
                loss = __uint_as_float(0x7FC00000u);
                atomicAdd(&status->bad_labels, 1);
            } else if (cls == 0) {
                const float* x = tile + threadIdx.x * pitch;
                float m = x[0];
                for (int j = 1; j < C; ++j) m = fmaxf(m, x[j]);
                const RowScale rs(m);
                float s = 0.f;
                int n_max = 0;
                for (int j = 0; j < C; ++j) {
                    const float v = x[j];
                    if (v < m) s += ex2(fmaf(v, kLog2e, rs.nml));
                    else ++n_max;
                }
                loss = finish_loss(m, x[static_cast<int>(y)], s, n_max, rs);
            }
            row_loss[row] = loss;
            h.add(loss);
        }
    }
    __syncthreads();
    h.flush();
}

// ---------------------------------------------------------------------------
// Short rows: one warp per row.  The warp reads the 16-byte-aligned superset of
// the row (VPL vectors per lane, all loads in flight together), masks what lies
// outside the row with -inf and keeps the row in registers for both passes.
// ---------------------------------------------------------------------------
constexpr int kWarpThreads = 256;

template <typename T, int VPL>
__global__ void __launch_bounds__(kWarpThreads)
score_warp_rows_kernel(const T* __restrict__ logits, const int64_t* __restrict__ labels, int64_t rows, int C,
                       int64_t ignore_index, float* __restrict__ row_loss, StatusBlock* status, uint32_t* hist0) {
    constexpr int EPV = Elem<T>::kPerVec;
    __shared__ uint32_t hist_s[kSelBins];
    Hist0 h{hist_s, hist0};
    h.clear();
    __syncthreads();
    const int lane = threadIdx.x & 31;
    const int64_t warps = static_cast<int64_t>(gridDim.x) * (kWarpThreads / 32);
    const int64_t row_bytes = static_cast<int64_t>(C) * sizeof(T);
    for (int64_t row = static_cast<int64_t>(blockIdx.x) * (kWarpThreads / 32) + (threadIdx.x >> 5); row < rows;
         row += warps) {
        const int64_t y = labels[row];
        const int cls = label_class(y, C, ignore_index);
        float loss = 0.f;
        if (cls == 2) {
            loss = __uint_as_float(0x7FC00000u);
            if (lane == 0) atomicAdd(&status->bad_labels, 1);
        } else if (cls == 0) {
            const uintptr_t ga = reinterpret_cast<uintptr_t>(logits) + row * row_bytes;
            const int head = static_cast<int>(ga & 15);
            const uint4* vbase = reinterpret_cast<const uint4*>(ga - head);
            const int nvec = static_cast<int>((head + row_bytes + 15) >> 4);
            const int e0 = -head / static_cast<int>(sizeof(T));  // element index of slot 0 of vector 0
            uint4 raw[VPL];
#pragma unroll
            for (int u = 0; u < VPL; ++u) {
                const int v = lane + 32 * u;
                raw[u] = v < nvec ? __ldcs(vbase + v) : make_uint4(0, 0, 0, 0);
            }
            const float xy = Elem<T>::widen(__ldg(logits + row * C + y));
            float x[VPL][EPV];
            float m = neg_inf();
#pragma unroll
            for (int u = 0; u < VPL; ++u) {
                const int j0 = e0 + (lane + 32 * u) * EPV;
                const uint32_t w[4] = {raw[u].x, raw[u].y, raw[u].z, raw[u].w};
#pragma unroll
                for (int e = 0; e < EPV; ++e) {
                    float v;
                    if constexpr (EPV == 4) v = __uint_as_float(w[e]);
                    else v = __uint_as_float((e & 1) ? (w[e >> 1] & 0xFFFF0000u) : (w[e >> 1] << 16));
                    const int j = j0 + e;
                    v = (j >= 0 && j < C) ? v : neg_inf();
                    x[u][e] = v;
                    m = fmaxf(m, v);
                }
            }
            m = warp_max(m);
            const RowScale rs(m);
            float s = 0.f;
            int n_max = 0;
#pragma unroll
            for (int u = 0; u < VPL; ++u)
#pragma unroll
                for (int e = 0; e < EPV; ++e) {
                    const float v = x[u][e];
                    if (v < m) s += ex2(fmaf(v, kLog2e, rs.nml));
                    else ++n_max;
                }
            s = warp_sum(s);
            n_max = warp_sum(n_max);
            loss = finish_loss(m, xy, s, n_max, rs);
        }
        if (lane == 0) {
            row_loss[row] = loss;
            h.add(loss);
        }
    }
    __syncthreads();
    h.flush();
}

// ---------------------------------------------------------------------------
// Long rows: one CTA per row, the row resident in shared memory.
// ---------------------------------------------------------------------------
constexpr int kCtaThreads = 256;
constexpr int kCtaWarps = kCtaThreads / 32;
constexpr uint32_t kBulkChunk = 16384;  // bytes per bulk copy

__device__ __forceinline__ uint32_t smem_u32(const void* p) { return static_cast<uint32_t>(__cvta_generic_to_shared(p)); }

__device__ __forceinline__ void mbar_init(uint64_t* bar, uint32_t count) {
    asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(smem_u32(bar)), "r"(count));
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
}
__device__ __forceinline__ void mbar_expect_tx(uint64_t* bar, uint32_t bytes) {
    asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(smem_u32(bar)), "r"(bytes) : "memory");
}
__device__ __forceinline__ bool mbar_try_wait(uint64_t* bar, uint32_t parity) {
    uint32_t ok;
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2, 2000;\n\t"
        "selp.u32 %0, 1, 0, p;\n\t}"
        : "=r"(ok)
        : "r"(smem_u32(bar)), "r"(parity)
        : "memory");
    return ok != 0;
}
// Bounded wait: false if the barrier did not flip within the poll limit.
__device__ __forceinline__ bool mbar_wait(uint64_t* bar, uint32_t parity) {
    for (uint32_t i = 0; i < kWaitLimit; ++i)
        if (mbar_try_wait(bar, parity)) return true;
    return false;
}
// 1-D bulk asynchronous copy global -> shared, completion counted in bytes on `bar`.
// dst, src 16-byte aligned; bytes a multiple of 16.
__device__ __forceinline__ void bulk_g2s(void* dst, const void* src, uint32_t bytes, uint64_t* bar) {
    asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];" ::"r"(
                     smem_u32(dst)),
                 "l"(src), "r"(bytes), "r"(smem_u32(bar))
                 : "memory");
}
__device__ __forceinline__ void fence_async_proxy() { asm volatile("fence.proxy.async.shared::cta;" ::: "memory"); }

struct CtaShared {
    uint64_t bar;
    int64_t row;      // row being processed, -1 = no more rows
    int32_t arg_pos;  // element position of the excluded maximum
    int32_t give_up;
    float red_f[kCtaWarps];
    int32_t red_i[kCtaWarps];
    float bcast;
};

template <typename T>
__global__ void __launch_bounds__(kCtaThreads)
score_cta_rows_kernel(const T* __restrict__ logits, const int64_t* __restrict__ labels, int64_t rows, int C,
                      int64_t ignore_index, float* __restrict__ row_loss, StatusBlock* status, uint32_t* hist0) {
    constexpr int EPV = Elem<T>::kPerVec;
    extern __shared__ __align__(128) unsigned char smem_raw[];
    CtaShared& sh = *reinterpret_cast<CtaShared*>(smem_raw);
    uint32_t* hist_s = reinterpret_cast<uint32_t*>(smem_raw + 128);
    unsigned char* buf = smem_raw + 128 + (hist0 ? kSelBins * sizeof(uint32_t) : 0);  // 128-byte aligned
    Hist0 h{hist_s, hist0};
    h.clear();
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const int64_t row_bytes = static_cast<int64_t>(C) * sizeof(T);
    if (tid == 0) {
        mbar_init(&sh.bar, 1);
        sh.give_up = 0;
    }
    __syncthreads();
    uint32_t parity = 0;

    for (;;) {
        // -- next row: a device-wide ticket, so that CTAs stay busy whatever the mask looks like
        if (tid == 0) {
            int64_t r;
            for (;;) {
                r = static_cast<int64_t>(atomicAdd(&status->row_ticket, 1u));
                if (r >= rows) {
                    r = -1;
                    break;
                }
                const int cls = label_class(labels[r], C, ignore_index);
                if (cls == 0) break;
                float l = 0.f;
                if (cls == 2) {
                    l = __uint_as_float(0x7FC00000u);
                    atomicAdd(&status->bad_labels, 1);
                }
                row_loss[r] = l;
                h.add(l);
            }
            sh.row = r;
            sh.arg_pos = 0x7FFFFFFF;
        }
        __syncthreads();  // also: every thread is done with the previous row's buffer
        const int64_t row = sh.row;
        if (row < 0 || sh.give_up) break;

        const uintptr_t ga = reinterpret_cast<uintptr_t>(logits) + row * row_bytes;
        const int head = static_cast<int>(ga & 15);
        const int nvec = static_cast<int>((head + row_bytes + 15) >> 4);
        const int first_body = head ? 1 : 0;                                   // vectors fully inside the row
        const int end_body = static_cast<int>((head + row_bytes) >> 4);
        if (tid == 0) {
            fence_async_proxy();  // earlier generic-proxy accesses of the buffer before the async writes
            const uint32_t body = static_cast<uint32_t>(end_body - first_body) << 4;
            mbar_expect_tx(&sh.bar, body);
            const unsigned char* src = reinterpret_cast<const unsigned char*>(ga - head) + (first_body << 4);
            unsigned char* dst = buf + (first_body << 4);
            for (uint32_t o = 0; o < body; o += kBulkChunk)
                bulk_g2s(dst + o, src + o, min(kBulkChunk, body - o), &sh.bar);
        } else if (tid >= 32 && tid < 32 + 2 * EPV) {
            // ragged head and tail: element loads, -inf outside the row
            const int slot = (tid - 32) % EPV;
            const bool tail = (tid - 32) >= EPV;
            const int v = tail ? end_body : 0;
            if ((tail && end_body < nvec) || (!tail && head)) {
                const int64_t j = (static_cast<int64_t>(v) * 16 - head) / static_cast<int>(sizeof(T)) + slot;
                T val = Elem<T>::neg_inf_elem();
                if (j >= 0 && j < C) val = logits[row * C + j];
                reinterpret_cast<T*>(buf)[v * EPV + slot] = val;
            }
        }
        float xy = 0.f;
        if (tid == 0) xy = Elem<T>::widen(__ldg(logits + row * C + labels[row]));
        if (!mbar_wait(&sh.bar, parity)) {
            // the copy did not land in time: flag it, give it one more bounded wait so that
            // nothing is still writing into shared memory when the CTA leaves, and stop
            atomicExch(&status->timeout, 1);
            mbar_wait(&sh.bar, parity);
            sh.give_up = 1;
        }
        parity ^= 1;
        __syncthreads();
        if (sh.give_up) break;

        // -- pass 1: maximum
        const uint4* vec = reinterpret_cast<const uint4*>(buf);
        float m;
        if constexpr (EPV == 4) {
            m = neg_inf();
            for (int v = tid; v < nvec; v += kCtaThreads) {
                const uint4 q = vec[v];
                m = fmaxf(fmaxf(m, fmaxf(__uint_as_float(q.x), __uint_as_float(q.y))),
                          fmaxf(__uint_as_float(q.z), __uint_as_float(q.w)));
            }
        } else {
            __nv_bfloat162 mm = __halves2bfloat162(Elem<T>::neg_inf_elem(), Elem<T>::neg_inf_elem());
            for (int v = tid; v < nvec; v += kCtaThreads) {
                const uint4 q = vec[v];
                const __nv_bfloat162 a = __hmax2(*reinterpret_cast<const __nv_bfloat162*>(&q.x),
                                                 *reinterpret_cast<const __nv_bfloat162*>(&q.y));
                const __nv_bfloat162 b = __hmax2(*reinterpret_cast<const __nv_bfloat162*>(&q.z),
                                                 *reinterpret_cast<const __nv_bfloat162*>(&q.w));
                mm = __hmax2(mm, __hmax2(a, b));
            }
            m = fmaxf(__low2float(mm), __high2float(mm));
        }
        const float my_max = m;
        m = warp_max(m);
        if (lane == 0) sh.red_f[warp] = m;
        __syncthreads();
        m = sh.red_f[0];
#pragma unroll
        for (int w = 1; w < kCtaWarps; ++w) m = fmaxf(m, sh.red_f[w]);

        // -- take one occurrence of the maximum (the first) out of the row
        if (my_max == m) {
            int pos = 0x7FFFFFFF;
            for (int v = tid; v < nvec && pos == 0x7FFFFFFF; v += kCtaThreads)
                for (int e = 0; e < EPV; ++e)
                    if (Elem<T>::widen(reinterpret_cast<const T*>(buf)[v * EPV + e]) == m) {
                        pos = v * EPV + e;
                        break;
                    }
            atomicMin(&sh.arg_pos, pos);
        }
        __syncthreads();
        if (tid == 0) reinterpret_cast<T*>(buf)[sh.arg_pos] = Elem<T>::neg_inf_elem();
        __syncthreads();

        // -- pass 2: sum of exponentials (everything left is <= m; -inf gives 0)
        const RowScale rs(m);
        float s0 = 0.f, s1 = 0.f, s2 = 0.f, s3 = 0.f;
        for (int v = tid; v < nvec; v += kCtaThreads) {
            const uint4 q = vec[v];
            if constexpr (EPV == 4) {
                s0 += ex2(fmaf(__uint_as_float(q.x), kLog2e, rs.nml));
                s1 += ex2(fmaf(__uint_as_float(q.y), kLog2e, rs.nml));
                s2 += ex2(fmaf(__uint_as_float(q.z), kLog2e, rs.nml));
                s3 += ex2(fmaf(__uint_as_float(q.w), kLog2e, rs.nml));
            } else {
                s0 += ex2(fmaf(__uint_as_float(q.x << 16), kLog2e, rs.nml));
                s1 += ex2(fmaf(__uint_as_float(q.x & 0xFFFF0000u), kLog2e, rs.nml));
                s2 += ex2(fmaf(__uint_as_float(q.y << 16), kLog2e, rs.nml));
                s3 += ex2(fmaf(__uint_as_float(q.y & 0xFFFF0000u), kLog2e, rs.nml));
                s0 += ex2(fmaf(__uint_as_float(q.z << 16), kLog2e, rs.nml));
                s1 += ex2(fmaf(__uint_as_float(q.z & 0xFFFF0000u), kLog2e, rs.nml));
                s2 += ex2(fmaf(__uint_as_float(q.w << 16), kLog2e, rs.nml));
                s3 += ex2(fmaf(__uint_as_float(q.w & 0xFFFF0000u), kLog2e, rs.nml));
            }
        }
        float s = warp_sum((s0 + s1) + (s2 + s3));
        if (lane == 0) sh.red_f[warp] = s;  // the two barriers above separate this from the reads of the maxima
        __syncthreads();
        if (tid == 0) {
            s = sh.red_f[0];
#pragma unroll
            for (int w = 1; w < kCtaWarps; ++w) s += sh.red_f[w];
            const float loss = finish_loss(m, xy, s, 1, rs);
            row_loss[row] = loss;
            h.add(loss);
        }
    }
    __syncthreads();
    h.flush();
}

// ---------------------------------------------------------------------------
// Rows too long for shared memory: one CTA per row, two passes over global
// memory with plain element loads.  A plain fallback, not a tuned path.
// ---------------------------------------------------------------------------
template <typename T>
__global__ void __launch_bounds__(kCtaThreads)
score_huge_rows_kernel(const T* __restrict__ logits, const int64_t* __restrict__ labels, int64_t rows, int64_t C,
                       int64_t ignore_index, float* __restrict__ row_loss, StatusBlock* status, uint32_t* hist0) {
    __shared__ float red_f[kCtaWarps];
    __shared__ int red_i[kCtaWarps];
    __shared__ uint32_t hist_s[kSelBins];
    Hist0 h{hist_s, hist0};
    h.clear();
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    for (int64_t row = blockIdx.x; row < rows; row += gridDim.x) {
        const int64_t y = labels[row];
        const int cls = label_class(y, C, ignore_index);
        float loss = 0.f;
        __syncthreads();
        if (cls == 2) {
            loss = __uint_as_float(0x7FC00000u);
            if (tid == 0) atomicAdd(&status->bad_labels, 1);
        } else if (cls == 0) {
            const T* x = logits + row * C;
            float m = neg_inf();
            for (int64_t j = tid; j < C; j += kCtaThreads) m = fmaxf(m, Elem<T>::widen(x[j]));
            m = warp_max(m);
            if (lane == 0) red_f[warp] = m;
            __syncthreads();
            m = red_f[0];
            for (int w = 1; w < kCtaWarps; ++w) m = fmaxf(m, red_f[w]);
            __syncthreads();
            const RowScale rs(m);
            float s = 0.f;
            int n_max = 0;
            for (int64_t j = tid; j < C; j += kCtaThreads) {
                const float v = Elem<T>::widen(x[j]);
                if (v < m) s += ex2(fmaf(v, kLog2e, rs.nml));
                else ++n_max;
            }
            s = warp_sum(s);
            n_max = warp_sum(n_max);
            if (lane == 0) {
                red_f[warp] = s;
                red_i[warp] = n_max;
            }
            __syncthreads();
            if (tid == 0) {
                s = red_f[0];
                n_max = red_i[0];
                for (int w = 1; w < kCtaWarps; ++w) {
                    s += red_f[w];
                    n_max += red_i[w];
                }
                loss = finish_loss(m, Elem<T>::widen(x[y]), s, n_max, rs);
            }
        }
        if (tid == 0) {
            row_loss[row] = loss;
            h.add(loss);
        }
    }
    __syncthreads();
    h.flush();
}

// ---------------------------------------------------------------------------
// Sequence mean: L_n = (sum of the unmasked token losses) / count, one warp per
// sample, lanes stride over t and combine in a fixed butterfly, so the result
// does not depend on the launch geometry.  0 when every token is ignored.
// ---------------------------------------------------------------------------
__global__ void __launch_bounds__(256)
seq_mean_kernel(const float* __restrict__ token_loss, const int64_t* __restrict__ labels, int64_t N, int64_t T,
                int64_t ignore_index, float* __restrict__ losses, uint32_t* hist0) {
    __shared__ uint32_t hist_s[kSelBins];
    Hist0 h{hist_s, hist0};
    h.clear();
    __syncthreads();
    const int lane = threadIdx.x & 31;
    const int64_t warps = static_cast<int64_t>(gridDim.x) * 8;
    for (int64_t n = static_cast<int64_t>(blockIdx.x) * 8 + (threadIdx.x >> 5); n < N; n += warps) {
        float s = 0.f;
        int cnt = 0;
        for (int64_t t = lane; t < T; t += 32)
            if (labels[n * T + t] != ignore_index) {
                s += token_loss[n * T + t];
                ++cnt;
            }
        s = warp_sum(s);
        cnt = warp_sum(cnt);
        if (lane == 0) {
            const float l = cnt ? s / static_cast<float>(cnt) : 0.f;
            losses[n] = l;
            h.add(l);
        }
    }
    __syncthreads();
    h.flush();
}

template <typename K>
int blocks_per_sm(K kernel, int threads, size_t smem) {
    int b = 0;
    if (cudaOccupancyMaxActiveBlocksPerMultiprocessor(&b, kernel, threads, smem) != cudaSuccess || b < 1) b = 1;
    return b;
}

constexpr size_t kMaxDynSmem = 227 * 1024;

template <typename T>
cudaError_t launch_rows(const T* logits, const int64_t* labels, int64_t rows, int64_t C, int64_t ignore_index,
                        float* row_loss, StatusBlock* status, uint32_t* hist0, cudaStream_t s) {
    const int sms = sm_count();
    const int64_t row_bytes = C * static_cast<int64_t>(sizeof(T));
    if (C <= kTinyMaxC) {
        const int64_t tiles = (rows + kTinyThreads - 1) / kTinyThreads;
        const int grid = static_cast<int>(std::min<int64_t>(tiles, static_cast<int64_t>(sms) * 8));
        score_tiny_rows_kernel<T><<<grid, kTinyThreads, 0, s>>>(logits, labels, rows, static_cast<int>(C),
                                                                 ignore_index, row_loss, status, hist0);
        return cudaGetLastError();
    }
    const int64_t need_vec = (row_bytes + 30) / 16;  // vectors of the aligned superset, worst alignment
    if (need_vec <= 256) {
        const int64_t want = (rows + 7) / 8;
        auto go = [&](auto kernel) {
            const int grid = static_cast<int>(std::min<int64_t>(want, static_cast<int64_t>(sms) * blocks_per_sm(kernel, kWarpThreads, 0)));
            kernel<<<grid, kWarpThreads, 0, s>>>(logits, labels, rows, static_cast<int>(C), ignore_index, row_loss,
                                                 status, hist0);
        };
        if (need_vec <= 32) go(score_warp_rows_kernel<T, 1>);
        else if (need_vec <= 64) go(score_warp_rows_kernel<T, 2>);
        else if (need_vec <= 128) go(score_warp_rows_kernel<T, 4>);
        else go(score_warp_rows_kernel<T, 8>);
        return cudaGetLastError();
    }
    const size_t smem = 128 + (hist0 ? kSelBins * sizeof(uint32_t) : 0) + static_cast<size_t>((row_bytes + 32 + 127) / 128 * 128);
    if (smem <= kMaxDynSmem) {
        cudaError_t e = cudaFuncSetAttribute(score_cta_rows_kernel<T>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                             static_cast<int>(kMaxDynSmem));
        if (e != cudaSuccess) return e;
        const int bps = blocks_per_sm(score_cta_rows_kernel<T>, kCtaThreads, smem);
        const int grid = static_cast<int>(std::min<int64_t>(rows, static_cast<int64_t>(sms) * bps));
        score_cta_rows_kernel<T><<<grid, kCtaThreads, smem, s>>>(logits, labels, rows, static_cast<int>(C),
                                                                  ignore_index, row_loss, status, hist0);
        return cudaGetLastError();
    }
    const int grid = static_cast<int>(std::min<int64_t>(rows, static_cast<int64_t>(sms) * 8));
    score_huge_rows_kernel<T><<<grid, kCtaThreads, 0, s>>>(logits, labels, rows, C, ignore_index, row_loss, status,
                                                            hist0);
    return cudaGetLastError();
}

}  // namespace

cudaError_t launch_score(const void* logits, lsgd_dtype dt, const int64_t* labels, int64_t N, int64_t T, int64_t C,
                         int64_t ignore_index, float* losses, const ScoreWorkspace& ws, uint32_t* hist0,
                         cudaStream_t s) {
    const int64_t rows = N * T;
    float* row_loss = T == 1 ? losses : ws.token_loss;
    uint32_t* row_hist = T == 1 ? hist0 : nullptr;
    cudaError_t e = dt == LSGD_F32
                        ? launch_rows(static_cast<const float*>(logits), labels, rows, C, ignore_index, row_loss,
                                      ws.status, row_hist, s)
                        : launch_rows(static_cast<const __nv_bfloat16*>(logits), labels, rows, C, ignore_index,
                                      row_loss, ws.status, row_hist, s);
    if (e != cudaSuccess || T == 1) return e;
    const int grid = static_cast<int>(std::min<int64_t>((N + 7) / 8, static_cast<int64_t>(sm_count()) * 8));
    seq_mean_kernel<<<grid, 256, 0, s>>>(ws.token_loss, labels, N, T, ignore_index, losses, hist0);
    return cudaGetLastError();
}

}  // namespace lsgd
