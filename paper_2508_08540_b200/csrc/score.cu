// Per-sample loss record (Algorithm 1: the step that stores the loss of every
// processed sample): softmax cross-entropy per row of the candidate pool, mean
// over the unmasked tokens of a sample.
//
// Every row is evaluated from the sum over the OTHER classes (the true class y is left out):
//     M = max_{j != y} x_j,   S = sum_{j != y} exp(x_j - M)
//     x_y >= M:  l = log1p(S exp(M - x_y))
//     x_y <  M:  l = (M - x_y) + log(S + exp(x_y - M))
// which equals the textbook  (m - x_y) + log(sum_j exp(x_j - m)),  but adds only positive terms: nothing cancels,
// so losses near zero (a dominant true class) keep their relative accuracy in fp32, in a single pass and with no
// comparison per element.  exp(x_j - M) is evaluated as
//     ex2(fma(x_j, L, -fl(M L)))      with L = fl(log2 e),
// whose argument equals (x_j - M) L + d with d = fma(M, L, -fl(M L)) known exactly; the common factor 2^d
// cancels against the same rounded product in the last step (see loss_without_true_class).
//
// Row shapes and their kernels (all bound by the bytes of the logits):
//   short rows  (<= 416 B, or <= 32 elements)   one LANE per row: a warp copies 32 rows into its own shared-memory ring
//   small rows  (<= 2 KB)                        4, 8 or 16 lanes per row out of a block's shared-memory tile
//   medium rows (<= 256 KB)                      one warp per row, streamed through registers with a running (max, sum)
//   anything longer                              one CTA per row, two passes over global memory
// (rows of 417 bytes to 2 KB of a pool whose base is not 16-byte aligned are read element by element from the tile).
// Rows whose label is ignore_index are never scored; the kernels for medium and longer rows do not even
// read them (short and small rows are copied block-wise, ignored rows included).
#include <cuda_bf16.h>

#include <algorithm>
#include <mutex>
#include <type_traits>
#include <vector>

#include "lsgd_internal.cuh"

namespace lsgd {

namespace {

constexpr float kLog2e = 1.4426950408889634f;

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

// The selector's first radix digit, accumulated per CTA in shared memory (or, with smem == nullptr, added
// straight to the global histogram: kernels whose rows are long enough for one global atomic per row to be free).
struct Hist0 {
    uint32_t* smem;
    uint32_t* global;
    __device__ void clear() {
        if (global && smem)
            for (int i = threadIdx.x; i < kSelBins; i += blockDim.x) smem[i] = 0;
    }
    __device__ void add(float loss) {
        if (global) atomicAdd(smem ? &smem[loss_key(loss) >> 21] : &global[loss_key(loss) >> 21], 1u);
    }
    __device__ void flush() {
        if (global && smem)
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
// Vector arithmetic shared by the kernels for small and medium rows, and the loss
// formula they end in.
// ---------------------------------------------------------------------------
// Running maximum over vectors: packed bf16 pairs for bf16 rows (exact: a maximum rounds nothing).
template <typename T>
struct VecMax;
template <>
struct VecMax<float> {
    float m;
    __device__ VecMax() : m(neg_inf()) {}
    __device__ void add(const uint4& q) {
        m = fmaxf(fmaxf(m, fmaxf(__uint_as_float(q.x), __uint_as_float(q.y))),
                  fmaxf(__uint_as_float(q.z), __uint_as_float(q.w)));
    }
    __device__ float get() const { return m; }
};
template <>
struct VecMax<__nv_bfloat16> {
    __nv_bfloat162 m;
    __device__ VecMax() : m(__halves2bfloat162(__ushort_as_bfloat16(0xFF80u), __ushort_as_bfloat16(0xFF80u))) {}
    __device__ void add(const uint4& q) {
        const __nv_bfloat162 a = __hmax2(*reinterpret_cast<const __nv_bfloat162*>(&q.x),
                                         *reinterpret_cast<const __nv_bfloat162*>(&q.y));
        const __nv_bfloat162 b = __hmax2(*reinterpret_cast<const __nv_bfloat162*>(&q.z),
                                         *reinterpret_cast<const __nv_bfloat162*>(&q.w));
        m = __hmax2(m, __hmax2(a, b));
    }
    __device__ float get() const { return fmaxf(__low2float(m), __high2float(m)); }
};

// The two fp32 values a 32-bit word of the row holds (one for fp32 rows).
template <typename T>
__device__ __forceinline__ float word_lo(uint32_t w) {
    return sizeof(T) == 4 ? __uint_as_float(w) : __uint_as_float(w << 16);
}
__device__ __forceinline__ float word_hi(uint32_t w) { return __uint_as_float(w & 0xFFFF0000u); }

// Packed pairs of fp32 (Blackwell's two-wide fp32 FMA and add).
struct F2 {
    unsigned long long v;
};
__device__ __forceinline__ F2 pack2(float lo, float hi) {
    F2 r;
    asm("mov.b64 %0, {%1, %2};" : "=l"(r.v) : "f"(lo), "f"(hi));
    return r;
}
__device__ __forceinline__ void unpack2(F2 a, float& lo, float& hi) {
    asm("mov.b64 {%0, %1}, %2;" : "=f"(lo), "=f"(hi) : "l"(a.v));
}
__device__ __forceinline__ F2 fma2(F2 a, F2 b, F2 c) {
    F2 r;
    asm("fma.rn.f32x2 %0, %1, %2, %3;" : "=l"(r.v) : "l"(a.v), "l"(b.v), "l"(c.v));
    return r;
}
__device__ __forceinline__ F2 add2(F2 a, F2 b) {
    F2 r;
    asm("add.rn.f32x2 %0, %1, %2;" : "=l"(r.v) : "l"(a.v), "l"(b.v));
    return r;
}

// acc += 2^d exp(x - m) for a pair of elements: one two-wide FMA, two ex2, one two-wide add.
__device__ __forceinline__ void pair_sum_exp(float x0, float x1, F2 l2e, F2 nml, F2& acc) {
    float t0, t1;
    unpack2(fma2(pack2(x0, x1), l2e, nml), t0, t1);
    acc = add2(acc, pack2(ex2(t0), ex2(t1)));
}

// a0, a1 += 2^d exp(x - m) over the elements of one vector, in a fixed order.
template <typename T>
__device__ __forceinline__ void vec_sum_exp(const uint4& q, F2 l2e, F2 nml, F2& a0, F2& a1) {
    if constexpr (sizeof(T) == 4) {
        pair_sum_exp(__uint_as_float(q.x), __uint_as_float(q.y), l2e, nml, a0);
        pair_sum_exp(__uint_as_float(q.z), __uint_as_float(q.w), l2e, nml, a1);
    } else {
        pair_sum_exp(word_lo<T>(q.x), word_hi(q.x), l2e, nml, a0);
        pair_sum_exp(word_lo<T>(q.y), word_hi(q.y), l2e, nml, a1);
        pair_sum_exp(word_lo<T>(q.z), word_hi(q.z), l2e, nml, a0);
        pair_sum_exp(word_lo<T>(q.w), word_hi(q.w), l2e, nml, a1);
    }
}

// Sets slot e of a vector to -inf.
template <typename T>
__device__ __forceinline__ uint32_t blank_word(uint32_t w, int i, int e) {
    if constexpr (sizeof(T) == 4) return i == e ? 0xFF800000u : w;
    else return i != (e >> 1) ? w : (e & 1) ? ((w & 0x0000FFFFu) | 0xFF800000u) : ((w & 0xFFFF0000u) | 0x0000FF80u);
}
template <typename T>
__device__ __forceinline__ void blank_slot(uint4& q, int e) {
    q.x = blank_word<T>(q.x, 0, e);
    q.y = blank_word<T>(q.y, 1, e);
    q.z = blank_word<T>(q.z, 2, e);
    q.w = blank_word<T>(q.w, 3, e);
}

// The loss from the sum over the OTHER classes.  With M = max_{j != y} x_j, P = fl(M L) and
// S = sum_{j != y} 2^(x_j L - P) (= 2^D sum_{j != y} exp(x_j - M), D = M L - P; S = 0 if there is no other class):
//   x_y >= M:  l = log1p(u),  u = sum_{j != y} exp(x_j - x_y) = S 2^(P - x_y L)            (one fused multiply-add)
//   x_y <  M:  l = (M - x_y) + log(sum_j exp(x_j - M)) = (M - x_y) + log((S + 2^(x_y L - P)) 2^-D)
// Only sums of positive terms: nothing cancels, so a loss of 1e-9 is as accurate as a loss of 10, in one pass and
// without a comparison per element (a small loss means that the true class dominates, so it is the true class, not
// the maximum, that has to stay out of the sum).
// Both forms are evaluated without a branch and one is selected: log1p(u) as its series up to u^6 below 1/8
// (truncation 5e-7 relative) and as lg2(1 + u) ln 2 above (lg2.approx: 2^-22 absolute on a result above 0.11);
// the second form's loss is above ln 2, where the same absolute error is 3e-7 relative.
__device__ __forceinline__ float lg2(float x) {
    float y;
    asm("lg2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
    return y;
}
__device__ __forceinline__ float loss_without_true_class(float M, float P, float S, float xy) {
    constexpr float kLn2 = 0.6931471805599453f;
    const float u = S * ex2(fmaf(-xy, kLog2e, P));
    float series = fmaf(u, -1.0f / 6.0f, 0.2f);
    series = fmaf(u, series, -0.25f);
    series = fmaf(u, series, 1.0f / 3.0f);
    series = fmaf(u, series, -0.5f);
    series = fmaf(u, series, 1.0f);
    const float confident = u < 0.125f ? u * series : lg2(1.0f + u) * kLn2;
    const float D = fmaf(M, kLog2e, -P);
    const float other = (M - xy) + (lg2(S + ex2(fmaf(xy, kLog2e, -P))) - D) * kLn2;
    return xy >= M ? confident : other;
}

constexpr int kTinyThreads = 256;
constexpr int kTinyMaxC = 32;
constexpr int kTinyStages = 3;

__device__ __forceinline__ void cp_async16(void* smem_dst, const void* gsrc) {
    asm volatile("cp.async.cg.shared.global [%0], [%1], 16;" ::"r"(static_cast<uint32_t>(__cvta_generic_to_shared(smem_dst))),
                 "l"(gsrc)
                 : "memory");
}
__device__ __forceinline__ void cp_async_commit() { asm volatile("cp.async.commit_group;" ::: "memory"); }
template <int PENDING>
__device__ __forceinline__ void cp_async_wait() {
    asm volatile("cp.async.wait_group %0;" ::"n"(PENDING) : "memory");
}

// Bulk asynchronous copies (the TMA unit, untiled form) with completion counted on a shared-memory barrier:
// one instruction moves a whole tile, where 16-byte cp.async needs one instruction and an address per 16 bytes.
// Source and destination must be 16-byte aligned and the size a multiple of 16 bytes.
__device__ __forceinline__ uint32_t smem_addr(const void* p) { return static_cast<uint32_t>(__cvta_generic_to_shared(p)); }
__device__ __forceinline__ void mbar_init(uint64_t* bar, uint32_t arrivals) {
    asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(smem_addr(bar)), "r"(arrivals) : "memory");
}
__device__ __forceinline__ void mbar_expect_tx(uint64_t* bar, uint32_t bytes) {
    asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(smem_addr(bar)), "r"(bytes) : "memory");
}
__device__ __forceinline__ void bulk_copy(void* smem_dst, const void* gsrc, uint32_t bytes, uint64_t* bar) {
    asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];" ::"r"(smem_addr(smem_dst)),
                 "l"(gsrc), "r"(bytes), "r"(smem_addr(bar))
                 : "memory");
}
__device__ __forceinline__ bool mbar_try_wait(uint64_t* bar, uint32_t parity) {
    uint32_t ok;
    asm volatile(
        "{\n\t.reg .pred p;\n\tmbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\tselp.u32 %0, 1, 0, p;\n\t}"
        : "=r"(ok)
        : "r"(smem_addr(bar)), "r"(parity)
        : "memory");
    return ok != 0;
}
// Orders this thread's earlier generic-proxy accesses to shared memory before later asynchronous-proxy ones.
__device__ __forceinline__ void fence_proxy_async() { asm volatile("fence.proxy.async.shared::cta;" ::: "memory"); }

// ---------------------------------------------------------------------------
// Small rows (417 bytes to 2 KB): a CTA copies a tile of consecutive rows (one
// contiguous, 16-byte-aligned-superset byte range) into shared memory with
// vector loads; groups of L lanes then own one row each and read it from there.
// One warp per row would spend most of its instructions on 32-lane reductions
// and on the per-row epilogue; with L lanes per row those are shared by 32 / L
// rows.  Rows start on 16-, 8- or 4-byte boundaries according to their length and
// to the pool's offset from a 16-byte boundary (every tile starts at that offset),
// and a lane reads chunks of that size, l, l + L, ... of its row; rows that start on
// odd 2-byte boundaries are read element by element.
// ---------------------------------------------------------------------------
constexpr int kGroupThreads = 128;
constexpr int kGroupMaxRowBytes = 2048;
constexpr int kGroupStages = 2;
constexpr uint32_t kBulkWaitTries = 1u << 22;  // polls of a tile's barrier before the block gives up

// A chunk: the CB bytes (16, 8 or 4) a lane reads from shared memory at once, CB / sizeof(T) elements.
template <int CB>
struct ChunkWord;
template <>
struct ChunkWord<16> { using type = uint4; };
template <>
struct ChunkWord<8> { using type = uint2; };
template <>
struct ChunkWord<4> { using type = uint32_t; };

template <typename T, int CB>
__device__ __forceinline__ void unpack_chunk(const typename ChunkWord<CB>::type& q, float (&v)[CB / static_cast<int>(sizeof(T))]) {
    uint32_t w[CB / 4];
    if constexpr (CB == 16) { w[0] = q.x; w[1] = q.y; w[2] = q.z; w[3] = q.w; }
    else if constexpr (CB == 8) { w[0] = q.x; w[1] = q.y; }
    else { w[0] = q; }
    if constexpr (sizeof(T) == 4) {
#pragma unroll
        for (int e = 0; e < CB / 4; ++e) v[e] = __uint_as_float(w[e]);
    } else {
#pragma unroll
        for (int e = 0; e < CB / 4; ++e) {  // bf16 is the upper half of an fp32
            v[2 * e] = __uint_as_float(w[e] << 16);
            v[2 * e + 1] = __uint_as_float(w[e] & 0xFFFF0000u);
        }
    }
}

// Maximum of a chunk's elements (bf16: on packed pairs, before widening) and its contribution to
// sum 2^(x L - P) (two-wide FMAs and adds), for chunks of 16, 8 or 4 bytes.
template <typename T, int CB>
__device__ __forceinline__ float chunk_max(const typename ChunkWord<CB>::type& q) {
    uint32_t w[CB / 4];
    if constexpr (CB == 16) { w[0] = q.x; w[1] = q.y; w[2] = q.z; w[3] = q.w; }
    else if constexpr (CB == 8) { w[0] = q.x; w[1] = q.y; }
    else { w[0] = q; }
    if constexpr (sizeof(T) == 4) {
        float m = __uint_as_float(w[0]);
#pragma unroll
        for (int e = 1; e < CB / 4; ++e) m = fmaxf(m, __uint_as_float(w[e]));
        return m;
    } else {
        __nv_bfloat162 m = *reinterpret_cast<const __nv_bfloat162*>(&w[0]);
#pragma unroll
        for (int e = 1; e < CB / 4; ++e) m = __hmax2(m, *reinterpret_cast<const __nv_bfloat162*>(&w[e]));
        return fmaxf(__low2float(m), __high2float(m));
    }
}
// A chunk of -inf elements, and a running maximum over chunks (bf16: on packed pairs, widened once at the end).
template <typename T, int CB>
__device__ __forceinline__ typename ChunkWord<CB>::type chunk_fill() {
    constexpr uint32_t f = sizeof(T) == 4 ? 0xFF800000u : 0xFF80FF80u;
    if constexpr (CB == 16) return make_uint4(f, f, f, f);
    else if constexpr (CB == 8) return make_uint2(f, f);
    else return f;
}
template <typename T>
struct ChunkMax;
template <>
struct ChunkMax<float> {
    float m;
    __device__ ChunkMax() : m(neg_inf()) {}
    __device__ __forceinline__ void word(uint32_t w) { m = fmaxf(m, __uint_as_float(w)); }
    template <int CB>
    __device__ __forceinline__ void add(const typename ChunkWord<CB>::type& q) {
        if constexpr (CB == 16) { word(q.x); word(q.y); word(q.z); word(q.w); }
        else if constexpr (CB == 8) { word(q.x); word(q.y); }
        else word(q);
    }
    __device__ __forceinline__ float get() const { return m; }
};
template <>
struct ChunkMax<__nv_bfloat16> {
    uint32_t m;
    __device__ ChunkMax() : m(0xFF80FF80u) {}
    __device__ __forceinline__ void word(uint32_t w) {
        const __nv_bfloat162 r = __hmax2(*reinterpret_cast<const __nv_bfloat162*>(&m), *reinterpret_cast<const __nv_bfloat162*>(&w));
        m = *reinterpret_cast<const uint32_t*>(&r);
    }
    template <int CB>
    __device__ __forceinline__ void add(const typename ChunkWord<CB>::type& q) {
        if constexpr (CB == 16) { word(q.x); word(q.y); word(q.z); word(q.w); }
        else if constexpr (CB == 8) { word(q.x); word(q.y); }
        else word(q);
    }
    __device__ __forceinline__ float get() const { return fmaxf(__uint_as_float(m << 16), __uint_as_float(m & 0xFFFF0000u)); }
};

template <typename T, int CB>
__device__ __forceinline__ void chunk_sum_exp(const typename ChunkWord<CB>::type& q, F2 l2e, F2 nml, F2& a0, F2& a1) {
    float v[CB / static_cast<int>(sizeof(T))];
    unpack_chunk<T, CB>(q, v);
    constexpr int n = CB / static_cast<int>(sizeof(T));  // 2, 4 or 8 elements
    pair_sum_exp(v[0], v[1], l2e, nml, a0);
    if constexpr (n >= 4) pair_sum_exp(v[2], v[3], l2e, nml, a1);
    if constexpr (n == 8) {
        pair_sum_exp(v[4], v[5], l2e, nml, a0);
        pair_sum_exp(v[6], v[7], l2e, nml, a1);
    }
}

// Tiles flow through a ring of kGroupStages buffers filled by asynchronous 16-byte copies (global -> shared, past
// the registers), one tile ahead of the one being reduced, so every CTA always has loads in flight; two stages
// rather than three leave room for a third CTA per SM, which is worth more (measured).
// REGS: a lane's share of the row (at most 128 bytes) is held in registers for both passes; otherwise both passes loop
// over shared memory.
template <typename T, int L, int CB, bool REGS>
__global__ void __launch_bounds__(kGroupThreads, 8)
score_group_rows_kernel(const T* __restrict__ logits, const int64_t* __restrict__ labels, int64_t rows, int C,
                        int64_t ignore_index, float* __restrict__ row_loss, StatusBlock* status, uint32_t* hist0,
                        int stage_bytes) {
    constexpr int R = kGroupThreads / L;  // rows per tile = lane groups per CTA
    constexpr bool VEC = CB > 0;          // rows start on CB-byte boundaries and are whole chunks
    constexpr bool PADDED = CB == 16 && L < 8;
    extern __shared__ __align__(16) unsigned char group_smem[];
    unsigned char* stages = group_smem;
    uint64_t* bars = reinterpret_cast<uint64_t*>(group_smem + kGroupStages * stage_bytes);  // a tile has landed: one per stage
    if (threadIdx.x == 0) {
#pragma unroll
        for (int st = 0; st < kGroupStages; ++st) mbar_init(bars + st, 1);
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");  // the barriers are set up before any copy names them
    }
    __syncthreads();
    Hist0 h{nullptr, hist0};  // rows of more than 416 bytes: one global atomic per row costs nothing
    h.clear();
    const int row_bytes = C * static_cast<int>(sizeof(T));
    const int64_t tiles = (rows + R - 1) / R;
    const int g = threadIdx.x / L, l = threadIdx.x % L;
    // 16-byte chunks, L == 4: two rows share a quarter-warp's accesses, so rows are laid out in shared memory with
    // a pitch of 4 (mod 8) chunks, which puts neighbouring rows four bank groups apart whatever the row length.
    // (The order in which a row's elements are summed must not depend on where the row sits: copies of a row
    // have to score the same bits.)
    const int nchunk = VEC ? row_bytes / (VEC ? CB : 1) : 0;
    const int pitch_bytes = PADDED ? 16 * (nchunk + ((L - nchunk) & 7)) : row_bytes;
    const int64_t my_tiles = tiles > blockIdx.x ? (tiles - blockIdx.x + gridDim.x - 1) / gridDim.x : 0;

    // Requests this CTA's i-th tile into stage i % kGroupStages.  Rows at their natural pitch: ONE bulk copy of the
    // tile's 16-byte-aligned superset (every tile starts `head` bytes past a boundary; an aligned block that holds a
    // valid byte is safe to read in full), issued by one thread: against 16-byte cp.async from all threads, which
    // spend an instruction and an address per 16 bytes, bf16 rows of 600 to 2,000 bytes gained 0.76 -> 0.83, 0.79 -> 0.85
    // of the copy rate (same run) and fp32 rows of 2,000 bytes 0.97 -> 1.07.  Rows at a padded pitch (16-byte chunks on
    // 4 lanes) keep the cp.async copies, which place every chunk: one bulk copy per row of 512 to 800 bytes was slower
    // (0.97 -> 0.89).  The stage was last touched before the block-wide barrier that precedes this call.
    auto issue = [&](int64_t i) {
        if constexpr (PADDED) {
            if (i < my_tiles) {
                const int64_t row0 = (blockIdx.x + i * gridDim.x) * R;
                const int nrows = rows - row0 < R ? static_cast<int>(rows - row0) : R;
                const uint4* src = reinterpret_cast<const uint4*>(reinterpret_cast<uintptr_t>(logits) + row0 * row_bytes);
                const int nvec = (nrows * row_bytes) >> 4;
                uint4* dst = reinterpret_cast<uint4*>(stages + (i % kGroupStages) * stage_bytes);
                const float inv_nchunk = 1.0f / static_cast<float>(nchunk);
                for (int v = threadIdx.x; v < nvec; v += kGroupThreads) {
                    const int r = __float2int_rz((static_cast<float>(v) + 0.5f) * inv_nchunk);  // v / nchunk, exact here
                    cp_async16(dst + r * (pitch_bytes >> 4) + (v - r * nchunk), src + v);
                }
            }
            cp_async_commit();  // one group per tile slot, also when it is empty: the wait below counts groups
        } else {
            if (i >= my_tiles || threadIdx.x != 0) return;
            const int64_t row0 = (blockIdx.x + i * gridDim.x) * R;
            const int nrows = rows - row0 < R ? static_cast<int>(rows - row0) : R;
            const uintptr_t b0 = reinterpret_cast<uintptr_t>(logits) + row0 * row_bytes;
            const int head = static_cast<int>(b0 & 15);
            const uint32_t bytes = static_cast<uint32_t>((head + nrows * row_bytes + 15) >> 4) << 4;
            uint64_t* bar = bars + (i % kGroupStages);
            fence_proxy_async();
            mbar_expect_tx(bar, bytes);
            bulk_copy(stages + (i % kGroupStages) * stage_bytes, reinterpret_cast<const void*>(b0 - head), bytes, bar);
        }
    };
    // Waits for tile i (all threads poll; the limit is seconds, never reached by a copy that was issued).
    auto landed = [&](int64_t i) -> bool {
        uint64_t* bar = bars + (i % kGroupStages);
        const uint32_t parity = static_cast<uint32_t>(i / kGroupStages) & 1u;
        for (uint32_t tries = 0; tries < kBulkWaitTries; ++tries)
            if (mbar_try_wait(bar, parity)) return true;
        return false;
    };
    auto label_at = [&](int64_t row) -> int64_t {  // (a tile past this CTA's last one starts past the pool's end)
        return row < rows ? labels[row] : ignore_index;
    };

#pragma unroll
    for (int i = 0; i < kGroupStages - 1; ++i) issue(i);
    int64_t y = label_at(static_cast<int64_t>(blockIdx.x) * R + g);
    // every tile starts at the same offset from a 16-byte boundary (a tile's rows are a multiple of 16 bytes)
    const int head = static_cast<int>(reinterpret_cast<uintptr_t>(logits) & 15);
    const int64_t row_step = static_cast<int64_t>(gridDim.x) * R;
    int64_t row_use = static_cast<int64_t>(blockIdx.x) * R;
    grid_dependency_wait();  // the status block and the histogram are clear from here on (the first tiles are on their way)
    for (int64_t i = 0; i < my_tiles; ++i) {
        issue(i + kGroupStages - 1);
        const int64_t y_next = label_at(row_use + row_step + g);
        if constexpr (PADDED) {
            cp_async_wait<kGroupStages - 1>();
            __syncthreads();  // everybody's copies of tile i have landed
        } else if (__syncthreads_or(!landed(i))) {  // (never, see above) give up as one: report, let the copies in flight end, leave
            if (threadIdx.x == 0) atomicExch(&status->timeout, 1);
            landed(i);
            if (i + 1 < my_tiles) landed(i + 1);
            break;
        }
        const int64_t row0 = row_use;  // (blockIdx.x + i gridDim.x) R, kept as a running sum
        row_use += row_step;
        const bool mine = row0 + g < rows;
        unsigned char* buf = stages + (i % kGroupStages) * stage_bytes;
        const int cls = mine ? label_class(y, C, ignore_index) : 1;
        T* x = reinterpret_cast<T*>(buf + head + g * pitch_bytes);
        // the true class stays out of the sum (see loss_without_true_class): its slot is read, then blanked
        float xy = 0.f;
        if (cls == 0 && l == 0) {
            xy = Elem<T>::widen(x[static_cast<int>(y)]);
            x[static_cast<int>(y)] = Elem<T>::neg_inf_elem();
            if constexpr (!PADDED) fence_proxy_async();  // this write stays ahead of the bulk copy that refills the stage later
        }
        __syncwarp();
        float m = -1e30f, s = 0.f;
        if constexpr (VEC && REGS) {
            // A lane's share of a row is at most 128 bytes (the launcher gives this path rows of up to 1024 and 2048
            // bytes over 8 and 16 lanes, never longer ones): it is read from shared memory once, into registers,
            // and both passes run from there, fully unrolled.  Round i (chunks i L .. i L + L - 1) is skipped by the whole warp once it is past the row.
            constexpr int CBV = VEC ? CB : 16;
            constexpr int kMaxCh = 128 / CBV;
            using Word = typename ChunkWord<CBV>::type;
            const Word* xv = reinterpret_cast<const Word*>(x);
            const int nch = cls == 0 ? nchunk : 0;  // groups without a row to score run the reductions on nothing
            Word w[kMaxCh];
            ChunkMax<T> cm;
#pragma unroll
            for (int i = 0; i < kMaxCh; ++i) {
                if (i * L < nchunk) {  // the same for every thread of the CTA
                    const int c = l + i * L;
                    w[i] = c < nch ? xv[c] : chunk_fill<T, CBV>();
                    cm.template add<CBV>(w[i]);
                }
            }
            m = fmaxf(m, cm.get());
#pragma unroll
            for (int o = L / 2; o > 0; o >>= 1) m = fmaxf(m, __shfl_xor_sync(0xFFFFFFFFu, m, o));
            const float P = m * kLog2e;
            const F2 l2e = pack2(kLog2e, kLog2e), nml = pack2(-P, -P);
            F2 a0 = pack2(0.f, 0.f), a1 = pack2(0.f, 0.f);
#pragma unroll
            for (int i = 0; i < kMaxCh; ++i)
                if (i * L < nchunk) chunk_sum_exp<T, CBV>(w[i], l2e, nml, a0, a1);
            float t0, t1, t2, t3;
            unpack2(a0, t0, t1);
            unpack2(a1, t2, t3);
            s = (t0 + t1) + (t2 + t3);
        } else if constexpr (VEC) {
            // plain loops over the lane's chunks (4 lanes per row: measured faster than the unrolled register copy
            // above, whose fixed cost short rows do not repay; 8 lanes per row on rows of 1 to 1.75 KB: a lane's
            // share no longer fits 128 bytes, and half the lanes of the 16-lane variant still win)
            using Word = typename ChunkWord<VEC ? CB : 16>::type;
            const Word* xv = reinterpret_cast<const Word*>(x);
            const int nch = cls == 0 ? nchunk : 0;
#pragma unroll 4
            for (int c = l; c < nch; c += L) m = fmaxf(m, chunk_max<T, VEC ? CB : 16>(xv[c]));
#pragma unroll
            for (int o = L / 2; o > 0; o >>= 1) m = fmaxf(m, __shfl_xor_sync(0xFFFFFFFFu, m, o));
            const float P = m * kLog2e;
            const F2 l2e = pack2(kLog2e, kLog2e), nml = pack2(-P, -P);
            F2 a0 = pack2(0.f, 0.f), a1 = pack2(0.f, 0.f);
#pragma unroll 4
            for (int c = l; c < nch; c += L) chunk_sum_exp<T, VEC ? CB : 16>(xv[c], l2e, nml, a0, a1);
            float t0, t1, t2, t3;
            unpack2(a0, t0, t1);
            unpack2(a1, t2, t3);
            s = (t0 + t1) + (t2 + t3);
        } else {
            const int n = cls == 0 ? C : 0;
            for (int j = l; j < n; j += L) m = fmaxf(m, Elem<T>::widen(x[j]));
#pragma unroll
            for (int o = L / 2; o > 0; o >>= 1) m = fmaxf(m, __shfl_xor_sync(0xFFFFFFFFu, m, o));
            const float P = m * kLog2e;
            for (int j = l; j < n; j += L) s += ex2(fmaf(Elem<T>::widen(x[j]), kLog2e, -P));
        }
#pragma unroll
        for (int o = L / 2; o > 0; o >>= 1) s += __shfl_xor_sync(0xFFFFFFFFu, s, o);
        if (mine && l == 0) {
            float loss = 0.f;
            if (cls == 2) {
                loss = __uint_as_float(0x7FC00000u);
                atomicAdd(&status->bad_labels, 1);
            } else if (cls == 0) {
                loss = loss_without_true_class(m, m * kLog2e, s, xy);
            }
            row_loss[row0 + g] = loss;
            h.add(loss);
        }
        __syncthreads();  // the stage may be refilled
        y = y_next;
    }
    if constexpr (PADDED) cp_async_wait<0>();
    h.flush();
}

// ---------------------------------------------------------------------------
// Short rows (up to kLaneMaxRowBytes, or at most 32 elements): a WARP takes 32 consecutive rows (one contiguous
// byte range; 32 rows are a multiple of 16 bytes, so every block starts at the same offset `head` from a 16-byte
// boundary), brings their aligned superset into its own ring of shared-memory stages with 16-byte asynchronous copies, one or two blocks of rows ahead of the one being scored, and every LANE scores one row.
// Nothing in the loop synchronises more than a warp, and the per-row work (label, reductions, the logarithm) is
// done once per lane instead of once per group of lanes.  Rows that are whole 16-byte chunks (of an aligned pool)
// are laid out at an odd chunk pitch; other rows are copied flat and read in units of the largest power of two (8, 4
// or 2 bytes) that divides the row length and the offset `head`, so that the lanes' strides are odd multiples of the
// unit: no bank conflicts either way (except for whole-chunk rows of a misaligned pool, which are merely correct).
// CMAX > 0 (rows of at most 32 elements): the row is read once into CMAX registers (slots past C hold -inf).
// CMAX == 0: two passes over the row in shared memory (maximum, then the sum), in units of CB bytes.
// A row's sum runs over its elements in an order that depends on C only, so copies of a row score the same bits
// wherever they sit.
// ---------------------------------------------------------------------------
constexpr int kLaneThreads = 128;
constexpr int kLaneMaxRowBytes = 416;

template <typename T, int CMAX, int CB, int STAGES>
__global__ void __launch_bounds__(CMAX > 0 ? kTinyThreads : kLaneThreads)
score_lane_rows_kernel(const T* __restrict__ logits, const int64_t* __restrict__ labels, int64_t rows, int C,
                       int64_t ignore_index, float* __restrict__ row_loss, StatusBlock* status, uint32_t* hist0,
                       int stage_bytes, int head) {
    constexpr bool PADDED = CB == 16;  // (only with head == 0)
    constexpr int kWarpsPerCta = (CMAX > 0 ? kTinyThreads : kLaneThreads) / 32;
    constexpr int ES = static_cast<int>(sizeof(T));
    constexpr int EPC = 16 / ES;  // elements per 16-byte chunk
    extern __shared__ __align__(16) unsigned char lane_smem[];
    uint32_t* hist_s = reinterpret_cast<uint32_t*>(lane_smem);
    Hist0 h{hist_s, hist0};
    h.clear();
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    // (the histogram's 8 KB are only there when a histogram is asked for)
    unsigned char* ring = lane_smem + (hist0 ? kSelBins * sizeof(uint32_t) : 0) + static_cast<size_t>(warp) * STAGES * stage_bytes;
    const int row_bytes = C * ES;
    const int rc = PADDED ? row_bytes >> 4 : 1;  // chunks per row
    const int pitch = rc | 1;                     // odd: the eight lanes of a quarter-warp read eight different bank groups
    // Where the rows sit in the stage exactly as in memory (no padding chunk: every layout but whole-chunk rows of an
    // even number of chunks), a block of rows can be ONE bulk copy issued by lane 0, counted on the warp's own barrier
    // for that stage, instead of an instruction and an address per 16 bytes from every lane.  That pays where the
    // instruction stream is the limit (same run, of the copy rate: bf16 rows of 400 bytes 0.79 -> 0.87, of 100 bytes
    // 0.73 -> 0.77; fp32 rows of 40 bytes 0.80 -> 0.82, of 408 bytes 0.97 -> 1.05) and costs where memory is (fp32
    // rows of 400 bytes, whole chunks: 1.04 -> 0.97), so whole-chunk fp32 rows keep the 16-byte copies.
    // (fp32 rows read element by element lost too: C = 101 0.86 -> 0.78.)
    const bool flat = !PADDED ? !(ES == 4 && CMAX == 0 && CB == 4)
                              : (ES == 2 && CMAX == 0 ? (rc & 1) != 0 : false);  // (a constant in all but one case)
    uint64_t* bars = reinterpret_cast<uint64_t*>(lane_smem + (hist0 ? kSelBins * sizeof(uint32_t) : 0) +
                                                 static_cast<size_t>(kWarpsPerCta) * STAGES * stage_bytes) + warp * STAGES;
    const int64_t blocks = (rows + 31) >> 5;
    const int64_t gw = static_cast<int64_t>(blockIdx.x) * kWarpsPerCta + warp;
    const int64_t nw = static_cast<int64_t>(gridDim.x) * kWarpsPerCta;
    const int64_t mine = blocks > gw ? (blocks - gw + nw - 1) / nw : 0;
    const float inv_rc = 1.0f / static_cast<float>(rc);

    auto place = [&](int v) -> int {  // chunk v of a block of rows -> its chunk slot in the stage
        if constexpr (!PADDED) return v;
        const int r = __float2int_rz((static_cast<float>(v) + 0.5f) * inv_rc);  // v / rc, exact for v < 2^20
        return r * pitch + (v - r * rc);
    };
    // Running positions instead of i % STAGES, i / STAGES and i * nw on 64-bit values in every iteration (a division
    // by three alone is a dozen instructions, and a 40-byte row is worth about 270): same run, of the copy rate, fp32
    // C = 10 0.82 -> 0.89, bf16 C = 32 0.71 -> 0.75, bf16 C = 100 0.92 -> 0.95.  The memory-bound two-pass fp32 rows
    // keep the product for the row index: with the running sum they lost (C = 100: 1.04 -> 1.01).
    constexpr bool kRunningRows = CMAX > 0 || ES == 2;
    const int64_t row_step = nw << 5;
    int64_t n_iss = 0, row_iss = gw << 5, row_use = gw << 5;
    int s_iss = 0, s_use = 0;   // the stage of the next block to request / to score
    uint32_t parity = 0;        // bit s: the phase of stage s's barrier that the next wait on it waits for
    auto issue = [&]() -> int64_t {  // requests this warp's next block of rows; returns this lane's label
        int64_t y = ignore_index;
        if (n_iss < mine) {
            const int64_t row0 = kRunningRows ? row_iss : (gw + n_iss * nw) << 5;
            const int nrows = rows - row0 < 32 ? static_cast<int>(rows - row0) : 32;
            // the 16-byte-aligned superset of the block's bytes (every block starts `head` bytes past a boundary;
            // an aligned 16-byte unit that holds one valid byte is safe to read in full)
            const unsigned char* src = reinterpret_cast<const unsigned char*>(logits) + row0 * row_bytes - head;
            unsigned char* dst = ring + s_iss * stage_bytes;
            const int nvec = (head + nrows * row_bytes + 15) >> 4;
            if (flat) {
                if (lane == 0) {
                    fence_proxy_async();
                    mbar_expect_tx(bars + s_iss, static_cast<uint32_t>(nvec) << 4);
                    bulk_copy(dst, src, static_cast<uint32_t>(nvec) << 4, bars + s_iss);
                }
            } else {
                for (int v = lane; v < nvec; v += 32) cp_async16(dst + place(v) * 16, src + v * 16);
            }
            if (lane < nrows) y = labels[row0 + lane];
        }
        if (!flat) cp_async_commit();  // one group per slot, also when it is empty: the wait below counts groups
        ++n_iss;
        row_iss += row_step;
        s_iss = s_iss + 1 == STAGES ? 0 : s_iss + 1;
        return y;
    };
    if (lane == 0) {
#pragma unroll
        for (int st = 0; st < STAGES; ++st) mbar_init(bars + st, 1);
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    __syncthreads();  // the histogram is clear, the barriers are set up

    int64_t yq[STAGES > 1 ? STAGES - 1 : 1];  // labels of the blocks in flight
#pragma unroll
    for (int i = 0; i < STAGES - 1; ++i) yq[i] = issue();
    for (int64_t i = 0; i < mine; ++i) {
        const int64_t y_new = issue();
        int64_t y = y_new;  // STAGES == 1: no block ahead (pools so small that every warp gets at most one block)
        if constexpr (STAGES > 1) {
            y = yq[0];
#pragma unroll
            for (int q = 0; q + 1 < STAGES - 1; ++q) yq[q] = yq[q + 1];
            yq[STAGES - 2] = y_new;
        }
        if (flat) {
            bool ok = false;  // (the limit is seconds; a copy that was issued completes long before)
            for (uint32_t tries = 0; tries < kBulkWaitTries && !ok; ++tries) ok = mbar_try_wait(bars + s_use, (parity >> s_use) & 1u);
            if (!__all_sync(0xFFFFFFFFu, ok)) {
                grid_dependency_wait();  // (the status block is clear from here on)
                if (lane == 0) atomicExch(&status->timeout, 1);
                break;
            }
            parity ^= 1u << s_use;
        } else {
            cp_async_wait<STAGES - 1>();
            __syncwarp();  // every lane's copies of block i have landed
        }
        const int64_t row0 = kRunningRows ? row_use : (gw + i * nw) << 5;
        const bool valid = row0 + lane < rows;
        unsigned char* buf = ring + s_use * stage_bytes;
        row_use += row_step;
        s_use = s_use + 1 == STAGES ? 0 : s_use + 1;
        const int cls = valid ? label_class(y, C, ignore_index) : 1;
        T* rowe = reinterpret_cast<T*>(buf + (PADDED ? lane * pitch * 16 : head + lane * row_bytes));
        // the true class stays out of the sum (see loss_without_true_class): its slot is read, then blanked
        float xy = 0.f;
        if (cls == 0) {
            xy = Elem<T>::widen(rowe[static_cast<int>(y)]);
            rowe[static_cast<int>(y)] = Elem<T>::neg_inf_elem();
            if (flat) fence_proxy_async();  // this write stays ahead of the bulk copy that refills the stage later
        }
        float m = -1e30f, s = 0.f;
        if constexpr (CMAX > 0) {
            float x[CMAX];
            if constexpr (PADDED) {
                constexpr int kCh = CMAX / EPC;
                const uint4* rowv = reinterpret_cast<const uint4*>(rowe);
#pragma unroll
                for (int c = 0; c < kCh; ++c) {
                    if (c < rc) {
                        const uint4 q = rowv[c];
                        const uint32_t w[4] = {q.x, q.y, q.z, q.w};
#pragma unroll
                        for (int e = 0; e < 4; ++e) {
                            if constexpr (ES == 4) {
                                x[c * 4 + e] = __uint_as_float(w[e]);
                            } else {
                                x[c * 8 + 2 * e] = __uint_as_float(w[e] << 16);
                                x[c * 8 + 2 * e + 1] = __uint_as_float(w[e] & 0xFFFF0000u);
                            }
                        }
                    } else {
#pragma unroll
                        for (int e = 0; e < EPC; ++e) x[c * EPC + e] = neg_inf();
                    }
                }
            } else {
#pragma unroll
                for (int j = 0; j < CMAX; ++j) x[j] = j < C ? Elem<T>::widen(rowe[j]) : neg_inf();
            }
            __syncwarp();  // the stage may be refilled by the next issue
#pragma unroll
            for (int j = 0; j < CMAX; ++j) m = fmaxf(m, x[j]);
            const float P = m * kLog2e;
            const F2 l2e = pack2(kLog2e, kLog2e), nml = pack2(-P, -P);
            F2 acc = pack2(0.f, 0.f);
#pragma unroll
            for (int j = 0; j < CMAX; j += 2) pair_sum_exp(x[j], x[j + 1], l2e, nml, acc);
            float s0, s1;
            unpack2(acc, s0, s1);
            s = s0 + s1;
        } else if constexpr (CB * 2 > ES * 2 && CB >= 2 * ES) {
            // units of at least two elements: maximum on whole units (bf16: packed pairs), two-wide sums
            using Word = typename ChunkWord<CB>::type;
            const Word* xv = reinterpret_cast<const Word*>(rowe);
            const int nch = cls == 0 ? (PADDED ? rc : row_bytes / CB) : 0;
            ChunkMax<T> cm;
#pragma unroll 4
            for (int c = 0; c < nch; ++c) cm.template add<CB>(xv[c]);
            m = fmaxf(m, cm.get());
            const float P = m * kLog2e;
            const F2 l2e = pack2(kLog2e, kLog2e), nml = pack2(-P, -P);
            F2 a0 = pack2(0.f, 0.f), a1 = pack2(0.f, 0.f);
#pragma unroll 4
            for (int c = 0; c < nch; ++c) chunk_sum_exp<T, CB>(xv[c], l2e, nml, a0, a1);
            float t0, t1, t2, t3;
            unpack2(a0, t0, t1);
            unpack2(a1, t2, t3);
            s = (t0 + t1) + (t2 + t3);
            __syncwarp();
        } else {
            // single elements (rows of an odd number of elements)
            const int n = cls == 0 ? C : 0;
#pragma unroll 4
            for (int j = 0; j < n; ++j) m = fmaxf(m, Elem<T>::widen(rowe[j]));
            const float P = m * kLog2e;
#pragma unroll 4
            for (int j = 0; j < n; ++j) s += ex2(fmaf(Elem<T>::widen(rowe[j]), kLog2e, -P));
            __syncwarp();
        }
        float loss = 0.f;
        if (cls == 2) {
            loss = __uint_as_float(0x7FC00000u);
            grid_dependency_wait();  // the status block is clear from here on
            atomicAdd(&status->bad_labels, 1);
        } else if (cls == 0) {
            loss = loss_without_true_class(m, m * kLog2e, s, xy);
        }
        if (valid) {
            row_loss[row0 + lane] = loss;
            h.add(loss);
        }
    }
    cp_async_wait<0>();
    __syncthreads();
    grid_dependency_wait();  // the workspace's histogram is clear from here on
    h.flush();
}

// ---------------------------------------------------------------------------
// Medium rows (above 2 KB): one warp per row, the row streamed through
// registers in steps of kStreamU vectors per lane, the next step's loads in
// flight while the current one is reduced.  Each lane keeps a running maximum
// m_l and the sum s_l of 2^(x L - p_l), p_l = fl(m_l L), over its elements
// (L = log2 e; the true class is left out); a step that raises the maximum
// rescales s_l by 2^(p_old - p_new) (the difference of the two rounded products:
// exact whenever it matters).  At the end  S = sum_l s_l 2^(p_l - P),  P = fl(M L),
// M = max_l m_l.  Whole interior vectors need no masking; the partial vectors in
// which an unaligned row starts and ends are taken element by element.
// ---------------------------------------------------------------------------
constexpr int kStreamThreads = 256;
constexpr int kStreamU = 4;                       // vectors (16 bytes) per lane and step: 2 KB per warp and step
constexpr int kStreamMaxRowBytes = 256 * 1024;

template <typename T>
__global__ void __launch_bounds__(kStreamThreads)
score_stream_rows_kernel(const T* __restrict__ logits, const int64_t* __restrict__ labels, int64_t rows, int C,
                         int64_t ignore_index, float* __restrict__ row_loss, StatusBlock* status, uint32_t* hist0,
                         int batch) {
    constexpr int EPV = Elem<T>::kPerVec;
    constexpr int U = kStreamU;
    __shared__ uint32_t hist_s[kSelBins];
    Hist0 h{hist_s, hist0};
    h.clear();
    __syncthreads();
    const int lane = threadIdx.x & 31;
    const int64_t row_bytes = static_cast<int64_t>(C) * sizeof(T);
    const uint4 fill = make_uint4(0xFF80FF80u, 0xFF80FF80u, 0xFF80FF80u, 0xFF80FF80u);   // -inf in every bf16 slot
    const uint4 fill32 = make_uint4(0xFF800000u, 0xFF800000u, 0xFF800000u, 0xFF800000u);  // -inf in every fp32 slot
    const uint4 none = EPV == 4 ? fill32 : fill;
    // Rows are handed out in batches from a device-wide ticket (ignored rows cost nothing, so a fixed assignment
    // would leave warps idle at the end); a warp asks for its next batch before it starts on the current one.
    auto grab = [&]() -> int64_t {
        unsigned long long t = 0;
        if (lane == 0) t = atomicAdd(&status->stream_ticket, static_cast<unsigned long long>(batch));
        return static_cast<int64_t>(__shfl_sync(0xFFFFFFFFu, t, 0));
    };
    int64_t cur = grab(), ahead = grab();
    int64_t row = cur;
    int64_t y = row < rows ? labels[row] : ignore_index;
    while (row < rows) {
        // the row after this one: the next of the batch, else the first of the batch already granted
        const bool last_of_batch = row + 1 >= cur + batch || row + 1 >= rows;
        const int64_t row_next = last_of_batch ? ahead : row + 1;
        const int64_t y_next = row_next < rows ? labels[row_next] : ignore_index;  // requested a row ahead
        const int cls = label_class(y, C, ignore_index);
        float loss = 0.f;
        if (cls == 2) {
            loss = __uint_as_float(0x7FC00000u);
            if (lane == 0) atomicAdd(&status->bad_labels, 1);
        } else if (cls == 0) {
            const T* x_row = logits + row * C;
            const uintptr_t ga = reinterpret_cast<uintptr_t>(x_row);
            const int head = static_cast<int>(ga & 15);
            const uint4* vbase = reinterpret_cast<const uint4*>(ga - head);
            const int nvec = static_cast<int>((head + row_bytes + 15) >> 4);
            const int tail_bytes = static_cast<int>((head + row_bytes) & 15);  // bytes of the row in its last vector, 0 = all 16
            const int v_begin = head ? 1 : 0, v_end = tail_bytes ? nvec - 1 : nvec;  // the whole vectors
            const int n_head = head ? (16 - head) / static_cast<int>(sizeof(T)) : 0;  // elements before them
            const int n_tail = tail_bytes / static_cast<int>(sizeof(T));              // elements after them
            const float xy = Elem<T>::widen(__ldg(x_row + y));

            // The true class is left out of the sum (its slot is blanked to -inf as its vector passes by), which is
            // all that the relative accuracy of tiny losses needs: see loss_without_true_class.
            const int y_byte = head + static_cast<int>(y) * static_cast<int>(sizeof(T));
            const int vy = y_byte >> 4;                                           // the vector that holds x_y ...
            const int ey = (y_byte & 15) / static_cast<int>(sizeof(T));           // ... and its slot there
            // Lane state: m (maximum so far), p = fl(m L), s = sum of 2^(x L - p) over the lane's elements so far.
            float m = -1e30f, p = -1e30f * kLog2e, s = 0.f;
            uint4 raw[U], nxt[U];
#pragma unroll
            for (int u = 0; u < U; ++u) {
                const int v = v_begin + u * 32 + lane;
                raw[u] = v < v_end ? __ldcg(vbase + v) : none;
            }
            for (int v0 = v_begin; v0 < v_end; v0 += 32 * U) {
#pragma unroll
                for (int u = 0; u < U; ++u) {  // the next step's vectors
                    const int v = v0 + 32 * U + u * 32 + lane;
                    nxt[u] = v < v_end ? __ldcg(vbase + v) : none;
                }
#pragma unroll
                for (int u = 0; u < U; ++u)
                    if (v0 + u * 32 + lane == vy) blank_slot<T>(raw[u], ey);
                {
                    VecMax<T> vm;  // bf16: the maximum is taken on packed pairs, before widening
#pragma unroll
                    for (int u = 0; u < U; ++u) vm.add(raw[u]);
                    const float mn = fmaxf(m, vm.get());
                    const float pn = mn * kLog2e;
                    s *= ex2(p - pn);  // the maximum rose: rescale (exactly 1 otherwise)
                    const F2 l2e = pack2(kLog2e, kLog2e), nml = pack2(-pn, -pn);
                    F2 a0 = pack2(0.f, 0.f), a1 = pack2(0.f, 0.f);  // two-wide FMAs and adds
#pragma unroll
                    for (int u = 0; u < U; ++u) vec_sum_exp<T>(raw[u], l2e, nml, a0, a1);
                    float t0, t1, t2, t3;
                    unpack2(a0, t0, t1);
                    unpack2(a1, t2, t3);
                    s += (t0 + t1) + (t2 + t3);
                    m = mn;
                    p = pn;
                }
#pragma unroll
                for (int u = 0; u < U; ++u) raw[u] = nxt[u];
            }
            if (n_head + n_tail > 0) {  // the partial vectors, one element per lane
                const int j = lane < n_head ? lane : lane < n_head + n_tail ? C - n_tail + (lane - n_head) : -1;
                const float v = (j >= 0 && j != static_cast<int>(y)) ? Elem<T>::widen(x_row[j]) : neg_inf();
                const float mn = fmaxf(m, v);
                const float pn = mn * kLog2e;
                s = s * ex2(p - pn) + ex2(fmaf(v, kLog2e, -pn));
                m = mn;
                p = pn;
            }
            const float M = warp_max(m);
            const float P = M * kLog2e;
            loss = loss_without_true_class(M, P, warp_sum(s * ex2(p - P)), xy);
        }
        if (lane == 0) {
            row_loss[row] = loss;
            h.add(loss);
        }
        y = y_next;
        row = row_next;
        if (last_of_batch) {
            cur = ahead;
            if (cur < rows) ahead = grab();
        }
    }
    __syncthreads();
    h.flush();
}

// ---------------------------------------------------------------------------
// Rows beyond 256 KB: one CTA per row, two passes over global memory with plain
// element loads.  A plain fallback, not a tuned path.
// ---------------------------------------------------------------------------
constexpr int kCtaThreads = 256;
constexpr int kCtaWarps = kCtaThreads / 32;

template <typename T>
__global__ void __launch_bounds__(kCtaThreads)
score_huge_rows_kernel(const T* __restrict__ logits, const int64_t* __restrict__ labels, int64_t rows, int64_t C,
                       int64_t ignore_index, float* __restrict__ row_loss, StatusBlock* status, uint32_t* hist0) {
    __shared__ float red_f[kCtaWarps];
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
            float m = -1e30f;  // maximum over the other classes (the true class stays out of the sum)
            for (int64_t j = tid; j < C; j += kCtaThreads)
                if (j != y) m = fmaxf(m, Elem<T>::widen(x[j]));
            m = warp_max(m);
            if (lane == 0) red_f[warp] = m;
            __syncthreads();
            m = red_f[0];
            for (int w = 1; w < kCtaWarps; ++w) m = fmaxf(m, red_f[w]);
            __syncthreads();
            const float P = m * kLog2e;
            float s = 0.f;
            for (int64_t j = tid; j < C; j += kCtaThreads)
                if (j != y) s += ex2(fmaf(Elem<T>::widen(x[j]), kLog2e, -P));
            s = warp_sum(s);
            if (lane == 0) red_f[warp] = s;
            __syncthreads();
            if (tid == 0) {
                s = red_f[0];
                for (int w = 1; w < kCtaWarps; ++w) s += red_f[w];
                loss = loss_without_true_class(m, P, s, Elem<T>::widen(x[y]));
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

// Resident blocks per multiprocessor of `kernel` at this block size and dynamic shared memory.  The answer (and
// the one-time opt-in to large dynamic shared memory) is remembered per device, kernel and size: the runtime calls
// behind it cost microseconds of host time, which a small pool's whole call is measured in.
template <typename K>
int blocks_per_sm(K kernel, int threads, size_t smem, bool large_smem = false) {
    struct Entry {
        const void* fn;
        int dev, threads, blocks;
        size_t smem;
    };
    static std::mutex mu;
    static std::vector<Entry> known;
    int dev = 0;
    cudaGetDevice(&dev);
    const void* fn = reinterpret_cast<const void*>(kernel);
    {
        std::lock_guard<std::mutex> lock(mu);
        for (const Entry& e : known)
            if (e.fn == fn && e.dev == dev && e.threads == threads && e.smem == smem) return e.blocks;
    }
    if (large_smem && cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, static_cast<int>(227 * 1024)) != cudaSuccess)
        return 0;
    int b = 0;
    if (cudaOccupancyMaxActiveBlocksPerMultiprocessor(&b, kernel, threads, smem) != cudaSuccess || b < 1) b = 1;
    std::lock_guard<std::mutex> lock(mu);
    known.push_back(Entry{fn, dev, threads, b, smem});
    return b;
}


template <typename T>
cudaError_t launch_rows(const T* logits, const int64_t* labels, int64_t rows, int64_t C, int64_t ignore_index,
                        float* row_loss, StatusBlock* status, uint32_t* hist0, cudaStream_t s) {
    const int sms = sm_count();
    const int64_t max_ctas = test_geometry().max_ctas;
    const int64_t row_bytes = C * static_cast<int64_t>(sizeof(T));
    if (C <= kTinyMaxC || row_bytes <= kLaneMaxRowBytes) {
        // one lane per row: the access unit is the largest power of two (at most 16 bytes) that divides the row
        // length and the pool's offset from a 16-byte boundary
        cudaError_t err = cudaSuccess;
        const int head = static_cast<int>(reinterpret_cast<uintptr_t>(logits) & 15);
        const int64_t both = row_bytes | head;
        const int cb = both % 16 == 0 ? 16 : both % 8 == 0 ? 8 : both % 4 == 0 ? 4 : 2;
        auto go = [&](auto kernel, int threads, int stages) {
            const int64_t rc = row_bytes / 16;
            const int stage_bytes = static_cast<int>(cb == 16 ? 32 * (rc | 1) * 16 : (head + 32 * row_bytes + 15) / 16 * 16);
            const size_t smem = (hist0 ? kSelBins * sizeof(uint32_t) : 0) + static_cast<size_t>(threads / 32) * stages * (stage_bytes + sizeof(uint64_t));  // rings + their barriers
            const int bps = blocks_per_sm(kernel, threads, smem, true);
            if (bps < 1) {
                err = cudaErrorInvalidValue;
                return;
            }
            const int64_t want = ((rows + 31) / 32 + threads / 32 - 1) / (threads / 32);
            const int grid = static_cast<int>(std::min({want, static_cast<int64_t>(sms) * bps, max_ctas}));
            // may start while the head of the workspace is still being cleared (the kernel waits before it touches it)
            err = launch_dependent_smem(kernel, grid, threads, smem, s, logits, labels, rows, static_cast<int>(C), ignore_index,
                                        row_loss, status, hist0, stage_bytes, head);
        };
        if (C <= kTinyMaxC) {
            auto by_len = [&](auto cb_tag) {
                constexpr int CBT = decltype(cb_tag)::value;  // 16: rows are whole chunks; 0: anything else
                constexpr bool f32 = sizeof(T) == 4;
                if (C <= 4) go(score_lane_rows_kernel<T, 4, f32 ? CBT : 0, kTinyStages>, kTinyThreads, kTinyStages);
                else if (C <= 8) go(score_lane_rows_kernel<T, 8, CBT, kTinyStages>, kTinyThreads, kTinyStages);
                else if (C <= 12) go(score_lane_rows_kernel<T, 12, f32 ? CBT : 0, kTinyStages>, kTinyThreads, kTinyStages);
                else if (C <= 16) go(score_lane_rows_kernel<T, 16, CBT, kTinyStages>, kTinyThreads, kTinyStages);
                else if (C <= 24) go(score_lane_rows_kernel<T, 24, CBT, kTinyStages>, kTinyThreads, kTinyStages);
                else go(score_lane_rows_kernel<T, 32, CBT, kTinyStages>, kTinyThreads, kTinyStages);
            };
            if (cb == 16) by_len(std::integral_constant<int, 16>{});
            else by_len(std::integral_constant<int, 0>{});
            return err;
        }
        auto by_unit = [&](auto stages_tag) {
            constexpr int ST = decltype(stages_tag)::value;
            if (cb == 16) go(score_lane_rows_kernel<T, 0, 16, ST>, kLaneThreads, ST);
            else if (cb == 8) go(score_lane_rows_kernel<T, 0, 8, ST>, kLaneThreads, ST);
            else if (cb == 4) go(score_lane_rows_kernel<T, 0, 4, ST>, kLaneThreads, ST);
            else go(score_lane_rows_kernel<T, 0, 2, ST>, kLaneThreads, ST);
        };
        // A pool so small that, with a single stage per warp, every block of 32 rows gets a warp of its own at once:
        // nothing to pipeline, and twice the warps are resident (a CIFAR-sized pool is scored in one wave).
        {
            const int64_t stage1 = cb == 16 ? 32 * ((row_bytes / 16) | 1) * 16 : (head + 32 * row_bytes + 15) / 16 * 16;
            const int64_t per_cta = (hist0 ? kSelBins * sizeof(uint32_t) : 0) + (kLaneThreads / 32) * stage1 + 1024;
            const int64_t ctas = std::min<int64_t>(32, (227 * 1024) / per_cta);
            if ((rows + 31) / 32 <= static_cast<int64_t>(sms) * ctas * (kLaneThreads / 32) && max_ctas >= static_cast<int64_t>(sms) * ctas) {
                by_unit(std::integral_constant<int, 1>{});
                return err;
            }
        }
        // warps per SM are what hides the latencies here, and the ring's size is what limits them: a third stage
        // only where sixteen warps still fit (measured: 176-byte rows lose a quarter going from 12 to 8 warps per SM)
        if (32 * row_bytes <= 4608) by_unit(std::integral_constant<int, 3>{});
        else by_unit(std::integral_constant<int, 2>{});
        return err;
    }
    if (row_bytes <= kGroupMaxRowBytes) {
        // the unit a lane reads: the largest power of two that divides the row length and the pool's offset from a
        // 16-byte boundary (every tile starts at that offset), 0 = single elements
        const int64_t both = row_bytes | static_cast<int64_t>(reinterpret_cast<uintptr_t>(logits) & 15);
        const int cb = both % 16 == 0 ? 16 : both % 8 == 0 ? 8 : both % 4 == 0 ? 4 : 0;
        cudaError_t err = cudaSuccess;
        auto go = [&](auto kernel, int lanes) {
            const int tile_rows = kGroupThreads / lanes;
            // bytes of one stage: the rows of a tile at their shared-memory pitch (rows of 16-byte chunks handled by
            // 4 lanes are padded to 4 (mod 8) chunks), or the flat copy of the tile's aligned superset
            const int64_t nchunk = row_bytes / 16;
            const int64_t pitch = (cb == 16 && lanes < 8) ? 16 * (nchunk + ((lanes - nchunk) & 7)) : row_bytes;
            const int stage_bytes = static_cast<int>((tile_rows * pitch + 32 + 15) / 16 * 16);
            const size_t smem = static_cast<size_t>(kGroupStages) * stage_bytes + kGroupStages * sizeof(uint64_t);  // stages + their barriers
            const int bps = blocks_per_sm(kernel, kGroupThreads, smem, true);
            if (bps < 1) {
                err = cudaErrorInvalidValue;
                return;
            }
            const int64_t tiles = (rows + tile_rows - 1) / tile_rows;
            const int grid = static_cast<int>(std::min({tiles, static_cast<int64_t>(sms) * bps, max_ctas}));
            err = launch_dependent_smem(kernel, grid, kGroupThreads, smem, s, logits, labels, rows, static_cast<int>(C), ignore_index,
                                        row_loss, status, hist0, stage_bytes);
        };
        auto by_chunk = [&](auto lanes_tag, auto regs_tag) {
            constexpr int LN = decltype(lanes_tag)::value;
            constexpr bool RG = decltype(regs_tag)::value;
            if (cb == 16) go(score_group_rows_kernel<T, LN, 16, RG>, LN);
            else if (cb == 8) go(score_group_rows_kernel<T, LN, 8, RG>, LN);
            else if (cb == 4 && sizeof(T) == 2) {
                if constexpr (sizeof(T) == 2) go(score_group_rows_kernel<T, LN, 4, RG>, LN);  // (4-byte chunks of fp32 are single elements)
            } else go(score_group_rows_kernel<T, LN, 0, false>, LN);
        };
        // rows per tile (128 / L) times bytes per row: at most 34 KB per stage (32 x 1024 at the padded pitch, 16 x 2048, 8 x 2048).
        // As few lanes per row as the row length allows: the per-row work is shared by the 32 / L rows of a warp.
        // Measured in one run, fraction of the copy rate: 600 and 800 bytes, 4 lanes 0.74-0.98 against 0.61-0.96 with
        // 8; 1000 bytes, 8 lanes (share in registers) 0.74 against 0.64 with 4 and 0.67 with 8 looping; 1280-1600
        // bytes, 8 lanes looping 0.86-1.02 against 0.71-0.97 with 16; 2000 bytes, fp32 1.00 with 8 lanes looping against
        // 0.94 with 16, bf16 (twice the elements per byte) 0.71 against 0.79.
        const bool vec = cb >= 8 || (cb == 4 && sizeof(T) == 2);
        if (row_bytes <= (sizeof(T) == 4 ? 1024 : 800)) by_chunk(std::integral_constant<int, 4>{}, std::false_type{});  // (fp32 1,024 bytes: 1.01 with 4 lanes, 0.97 with 8; bf16 0.79 against 0.86)
        else if (row_bytes <= 1024) by_chunk(std::integral_constant<int, 8>{}, std::true_type{});
        else if (row_bytes <= (sizeof(T) == 4 ? 2048 : 1792) && vec) by_chunk(std::integral_constant<int, 8>{}, std::false_type{});
        else by_chunk(std::integral_constant<int, 16>{}, std::true_type{});
        return err;
    }
    if (row_bytes <= kStreamMaxRowBytes) {
        const int64_t want = (rows + kStreamThreads / 32 - 1) / (kStreamThreads / 32);
        const int grid = static_cast<int>(std::min({
            want, static_cast<int64_t>(sms) * blocks_per_sm(score_stream_rows_kernel<T>, kStreamThreads, 0), max_ctas}));
        // rows per ticket: about 32 KB of logits
        const int batch = static_cast<int>(std::max<int64_t>(1, 32768 / row_bytes));
        score_stream_rows_kernel<T><<<grid, kStreamThreads, 0, s>>>(logits, labels, rows, static_cast<int>(C),
                                                                     ignore_index, row_loss, status, hist0, batch);
        return cudaGetLastError();
    }
    // longer rows are few per byte: a warp per row would leave most of the machine idle, so a CTA takes each
    const int grid = static_cast<int>(std::min({rows, static_cast<int64_t>(sms) * 8, max_ctas}));
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
    const int grid = static_cast<int>(std::min({(N + 7) / 8, static_cast<int64_t>(sm_count()) * 8, static_cast<int64_t>(test_geometry().max_ctas)}));
    seq_mean_kernel<<<grid, 256, 0, s>>>(ws.token_loss, labels, N, T, ignore_index, losses, hist0);
    return cudaGetLastError();
}

}  // namespace lsgd
