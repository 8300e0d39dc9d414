// Deterministic loss-based top-k selection (Section 4.2, "Data Allocation for
// Fast Workers": the highest-loss samples go to the fast workers).
//
// Total order: higher loss first, then lower index.  Losses are mapped to
// order-preserving 32-bit keys (loss_key), so everything below is integer work
// and the result is exact and bit-reproducible.
//
// One kernel does the whole selection, in phases separated by a barrier over all
// its thread blocks.  Pools above 65,536 entries (topk_select_kernel, a cooperative
// launch with one block per multiprocessor that exchanges through the workspace):
//   1. radix select: three digit histograms (11 + 11 + 10 bits, most significant
//      first; the first one may come ready-made from the scorer) find the key T of
//      the k-th entry and r, the number of entries equal to T that still belong to
//      the selection.  Every block resolves a digit for itself from the finished
//      histogram; a block keeps the keys of its first tile in registers throughout;
//   2. per-tile counts of keys above / equal to T (and the largest key);
//   3. ordered compaction: every key > T and the r lowest-index keys == T are
//      written in index order (scan-based positions: no atomics decide an order);
//   4. for loss-descending output, a stable LSD radix sort of the k (key, index)
//      pairs on u = (largest key - key) in 9-bit digits: only as many passes as
//      u's range needs (three for losses that span up to 16 binades above T, none
//      if all selected keys are equal); stability turns the index-ascending input
//      order into the required tie-break.  A pass is two phases: rank every tile
//      by the digit (which gives the tile's digit counts), then scatter.
//   All blocks are resident by construction; the barrier is an arrival counter in
//   the status block, polled with a limit: if it ever ran out, the block would set
//   the status block's timeout word and return, and the other blocks would follow.
// Pools of up to 65,536 entries run as ONE thread-block cluster whose barrier is the
// cluster's hardware barrier and which keeps its keys in registers and what blocks
// exchange in distributed shared memory: topk_cluster_kernel (index-ascending
// output: steps 1 to 3) and topk_cluster_sorted_kernel (loss-descending output:
// two digits of step 1, then a sort of every key from the k-th key's bin upwards
// with one barrier per pass; the first k sorted positions are the selection).
// Pools of at most kSmallN entries: loss-descending output by counting (small_rank_kernel: every entry counts the
// entries that come before it, no sort); index-ascending output from a single block that sorts the pool whole to
// find the k-th composite key (small_topk_kernel).
#include <cooperative_groups.h>

#include <algorithm>
#include <mutex>
#include <vector>

#include "lsgd_internal.cuh"

namespace lsgd {

// ---------------------------------------------------------------------------
// Geometry that the workspace layout depends on (host arithmetic only).
// ---------------------------------------------------------------------------
// Entries per sort tile: 1024 R with R in {1, 2, 4, 8}, the smallest that needs at most `max_tiles` tiles.
static int sort_rounds_for(int64_t k, int64_t max_tiles) {
    for (int r = 1; r < kSortMaxRounds; r <<= 1)
        if ((k + 1024 * r - 1) / (1024 * r) <= max_tiles) return r;
    return kSortMaxRounds;
}
// The same for the cooperative kernel, whose tiles need not be a power of two: any R from 1 to 8 (k = 320,000 on 148
// blocks: 105 tiles of 3,072 entries instead of 79 of 4,096).
static int sort_rounds_any(int64_t k, int64_t max_tiles) {
    for (int r = 1; r < kSortMaxRounds; ++r)
        if ((k + 1024 * r - 1) / (1024 * r) <= max_tiles) return r;
    return kSortMaxRounds;
}
// Upper bound of the number of sort tiles for any geometry the launcher may pick; grows with k, so that a
// workspace sized for k also serves every smaller k.
static size_t sort_tiles_bound(int64_t k) {
    if (k <= int64_t{kSortDirectTiles} * 1024 * kSortMaxRounds) return static_cast<size_t>(std::min<int64_t>(kSortDirectTiles, (k + 1023) / 1024));
    return static_cast<size_t>((k + 1024 * kSortMaxRounds - 1) / (1024 * kSortMaxRounds));
}
static size_t sort_count_words(int64_t k) { return sort_tiles_bound(k) * kSortBins; }

size_t topk_workspace_bytes(int64_t N, int64_t k) {
    if (N < 0 || k < 0 || k > N) return 0;
    const size_t tiles_n = static_cast<size_t>((N + kTile - 1) / kTile);
    size_t b = sizeof(StatusBlock);
    b += align_up(sizeof(uint32_t) * kSelPasses * kSelBins);
    b += align_up(sizeof(uint32_t) * sort_count_words(k));
    b += align_up(sizeof(uint32_t) * 4 * tiles_n);
    b += 4 * align_up(sizeof(uint32_t) * static_cast<size_t>(k));
    return b;
}

// Bytes at the start of the workspace that one memset must clear before a call: the status block and the
// selection's digit histograms.
static size_t topk_zero_bytes(int64_t) { return sizeof(StatusBlock) + align_up(sizeof(uint32_t) * kSelPasses * kSelBins); }

TopkWorkspace carve_topk(void* ws, int64_t N, int64_t k) {
    const size_t tiles_n = static_cast<size_t>((N + kTile - 1) / kTile);
    unsigned char* p = static_cast<unsigned char*>(ws);
    TopkWorkspace w;
    w.status = reinterpret_cast<StatusBlock*>(p);
    p += sizeof(StatusBlock);
    w.hist = reinterpret_cast<uint32_t*>(p);
    p += align_up(sizeof(uint32_t) * kSelPasses * kSelBins);
    w.tile_hist = reinterpret_cast<uint32_t*>(p);
    p += align_up(sizeof(uint32_t) * sort_count_words(k));
    w.tile_counts = reinterpret_cast<uint32_t*>(p);
    p += align_up(sizeof(uint32_t) * 4 * tiles_n);
    const size_t kb = align_up(sizeof(uint32_t) * static_cast<size_t>(k));
    w.pairs[0] = reinterpret_cast<uint2*>(p);
    w.pairs[1] = reinterpret_cast<uint2*>(p + 2 * kb);
    return w;
}

namespace {
__global__ void clear_words_kernel(uint4* p, int n) {
    grid_launch_dependents();
    const int i = blockIdx.x * blockDim.x + threadIdx.x;
    if (i < n) p[i] = make_uint4(0u, 0u, 0u, 0u);
}
}  // namespace

cudaError_t clear_device_words(void* p, size_t bytes, cudaStream_t s) {
    const int n = static_cast<int>(bytes / 16);
    clear_words_kernel<<<(n + 255) / 256, 256, 0, s>>>(static_cast<uint4*>(p), n);
    return cudaGetLastError();
}

cudaError_t zero_topk_workspace(void* ws, int64_t k, cudaStream_t s) { return clear_device_words(ws, topk_zero_bytes(k), s); }

namespace {

constexpr int kThreads = 1024;
constexpr int kWarps = kThreads / 32;
constexpr int kCounterPitch = kSortBins;      // one row of digit counters per warp
constexpr size_t kDynSmemBytes = sizeof(uint32_t) * kWarps * kCounterPitch;
constexpr uint32_t kMaxPolls = 1u << 21;      // barrier polls before a block gives up (seconds; never reached when all blocks are resident)

struct SelectParams {
    const float* losses;
    int64_t N;
    uint32_t k;
    int order;
    int32_t* out_idx;
    float* out_vals;
    TopkWorkspace ws;
    uint32_t sort_tiles;  // tiles of 1024 * sort_rounds entries over the k selected pairs
    int sort_rounds;
    int hist0_ready;      // the first digit's histogram was accumulated by the scorer
    uint32_t barrier_parties;  // blocks a barrier waits for: gridDim.x (a test hook adds one that never arrives)
    uint32_t barrier_polls;    // polls after which a block gives up
    int standalone;            // a selection on its own (no scorer before it in the call): the kernel resets the status block
};

__device__ __forceinline__ uint32_t digit_of(uint32_t key, int pass) {
    return pass == 0 ? key >> 21 : pass == 1 ? (key >> 10) & 0x7FFu : key & 0x3FFu;
}
__device__ __forceinline__ uint32_t prefix_mask(int pass) { return pass == 0 ? 0u : pass == 1 ? 0xFFE00000u : 0xFFFFFC00u; }

__device__ __forceinline__ uint32_t ld_acquire(const uint32_t* p) {
    uint32_t v;
    asm volatile("ld.acquire.gpu.u32 %0, [%1];" : "=r"(v) : "l"(p) : "memory");
    return v;
}

// Barrier over all blocks of a cooperatively launched kernel, with the other blocks' global writes visible
// afterwards (read them with __ldcg): an arrival counter that only grows; barrier number e is passed once
// e * gridDim.x arrivals are in.  Returns false if the wait ran out (or another block's did): the caller returns
// at once.
__device__ __forceinline__ bool grid_sync(StatusBlock* st, uint32_t& epoch, uint32_t parties, uint32_t max_polls) {
    __shared__ int ok_s;
    ++epoch;
    __syncthreads();
    if (threadIdx.x == 0) {
        const uint32_t target = epoch * parties;
        __threadfence();
        atomicAdd(&st->grid_arrivals, 1u);
        int ok = 1;
        uint32_t polls = 0;
        // (the acquiring load orders this thread's later reads, the block barrier below those of the other threads)
        while (ld_acquire(&st->grid_arrivals) < target) {
            if (++polls > max_polls || ((polls & 63u) == 0 && *reinterpret_cast<volatile int32_t*>(&st->timeout) != 0)) {
                ok = 0;
                break;
            }
            if (polls > 64u) __nanosleep(32);
        }
        if (!ok) atomicExch(&st->timeout, 1);
        ok_s = ok;
    }
    __syncthreads();
    return ok_s != 0;
}

// Block-wide exclusive scan of one value per thread.  `warp_tot` holds kWarps + 1 words; the block total is left
// in warp_tot[kWarps].
__device__ __forceinline__ uint32_t block_exclusive_scan(uint32_t v, uint32_t* warp_tot) {
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    uint32_t inc = v;
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) {
        const uint32_t n = __shfl_up_sync(0xFFFFFFFFu, inc, o);
        if (lane >= o) inc += n;
    }
    __syncthreads();  // warp_tot may still be read from an earlier call
    if (lane == 31) warp_tot[warp] = inc;
    __syncthreads();
    if (warp == 0) {
        const uint32_t w = warp_tot[lane];
        uint32_t wi = w;
#pragma unroll
        for (int o = 1; o < 32; o <<= 1) {
            const uint32_t n = __shfl_up_sync(0xFFFFFFFFu, wi, o);
            if (lane >= o) wi += n;
        }
        warp_tot[lane] = wi - w;
        if (lane == 31) warp_tot[kWarps] = wi;
    }
    __syncthreads();
    return warp_tot[warp] + inc - v;
}

// Walks a finished histogram from its highest bin down and finds the bin that holds the `want`-th entry (1-based).
// On return (all threads): bin, `want` reduced by the entries in the bins above it, and result[2] = the entries in
// the bin found (`result` holds three words).  Two block barriers: every warp scans the warps' totals for itself.
// `warp_tot` and `result` must not be written again before another block barrier has been passed (none is taken at
// the end).
template <bool GLOBAL>
__device__ __forceinline__ void find_bin(const uint32_t* hist, int nbins, uint32_t& want, uint32_t& bin, uint32_t* warp_tot, uint32_t* result) {
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    const bool two = nbins == 2 * kThreads;
    const int b0 = two ? nbins - 1 - 2 * static_cast<int>(threadIdx.x) : nbins - 1 - static_cast<int>(threadIdx.x);
    const uint32_t c0 = GLOBAL ? __ldcg(hist + b0) : hist[b0];
    const uint32_t c1 = !two ? 0u : GLOBAL ? __ldcg(hist + b0 - 1) : hist[b0 - 1];
    const uint32_t c = c0 + c1;
    uint32_t inc = c;
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) {
        const uint32_t n = __shfl_up_sync(0xFFFFFFFFu, inc, o);
        if (lane >= o) inc += n;
    }
    if (lane == 31) warp_tot[warp] = inc;
    __syncthreads();
    const uint32_t wt = warp_tot[lane];
    uint32_t winc = wt;
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) {
        const uint32_t n = __shfl_up_sync(0xFFFFFFFFu, winc, o);
        if (lane >= o) winc += n;
    }
    const uint32_t before = __shfl_sync(0xFFFFFFFFu, winc - wt, warp) + inc - c;
    if (before < want && want <= before + c) {
        const bool first = want <= before + c0;
        result[0] = first ? b0 : b0 - 1;
        result[1] = first ? want - before : want - before - c0;
        result[2] = first ? c0 : c1;
    }
    __syncthreads();
    bin = result[0];
    want = result[1];
}

// Loads the E keys a thread owns (consecutive indices from `base`), 0 beyond N.  Key 0 belongs to no loss
// (loss_key never returns it) and is below every threshold.
template <int E>
__device__ __forceinline__ void load_keys(const float* __restrict__ losses, int64_t N, int64_t base, uint32_t (&key)[E]) {
    if (base + E <= N && (reinterpret_cast<uintptr_t>(losses + base) & 15) == 0) {
        float4 q[E / 4];
#pragma unroll
        for (int i = 0; i < E / 4; ++i) q[i] = reinterpret_cast<const float4*>(losses + base)[i];
#pragma unroll
        for (int i = 0; i < E / 4; ++i) {
            key[4 * i] = loss_key(q[i].x);
            key[4 * i + 1] = loss_key(q[i].y);
            key[4 * i + 2] = loss_key(q[i].z);
            key[4 * i + 3] = loss_key(q[i].w);
        }
        return;
    }
#pragma unroll
    for (int i = 0; i < E; ++i) {
        const int64_t j = base + i;
        key[i] = j < N ? loss_key(losses[j]) : 0u;
    }
}

// Where each digit's run starts for a tile: base_s[d] = (entries of smaller digits, all tiles) + before_d.  Called by
// every thread of the block; thread d < kSortBins passes digit d's total over all tiles and its count in the tiles before
// this one, the others pass zeros.  `warp_sum` holds kSortBins / 32 words.
__device__ __forceinline__ void digit_bases(uint32_t total, uint32_t before, uint32_t* warp_sum, uint32_t* base_s) {
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    uint32_t inc = total;
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) {
        const uint32_t n = __shfl_up_sync(0xFFFFFFFFu, inc, o);
        if (lane >= o) inc += n;
    }
    if (tid < kSortBins && lane == 31) warp_sum[warp] = inc;
    __syncthreads();
    if (tid < kSortBins) {
        uint32_t below = 0;
#pragma unroll
        for (int w = 0; w < kSortBins / 32; ++w) below += w < warp ? warp_sum[w] : 0u;
        base_s[tid] = below + (inc - total) + before;
    }
    __syncthreads();
}

// The loss a key came from, where the key says it all; -0/+0 and NaNs (their sign and payload are not in the key) are
// read back from the table.
__device__ __forceinline__ float loss_of_key(uint32_t key, const float* __restrict__ losses, int32_t i) {
    if (key == 0x80000000u || key == 0xFFFFFFFFu) return losses[i];
    return __uint_as_float((key & 0x80000000u) ? key & 0x7FFFFFFFu : ~key);
}

// Lanes of the warp whose 9-bit digit equals this lane's, among the lanes with `live` set (0 for a lane that is
// not live).  Ten votes; cheaper here than the generic match instruction.
__device__ __forceinline__ uint32_t match_digit(uint32_t d, bool live) {
    uint32_t peers = __ballot_sync(0xFFFFFFFFu, live);
#pragma unroll
    for (int b = 0; b < kSortBits; ++b) {
        const bool bit = (d >> b) & 1u;
        const uint32_t m = __ballot_sync(0xFFFFFFFFu, bit);
        peers &= bit ? m : ~m;
    }
    return live ? peers : 0u;
}

// E: keys per thread of a selection tile (tiles of 1024 E entries, E = 4, 8, 12 or 16: the smallest that gives every
// tile a block of its own; block b takes tiles b, b + gridDim.x, ...).
template <int E>
__global__ void __launch_bounds__(kThreads, 1) topk_select_kernel(const __grid_constant__ SelectParams p) {
    extern __shared__ __align__(16) uint32_t dyn_smem[];  // selection: hist_s[kSelBins]; sort: counters[kWarps][kCounterPitch]
    __shared__ uint32_t warp_tot[kWarps + 1];
    __shared__ uint32_t result[3];
    __shared__ uint32_t red[3];
    __shared__ uint32_t part_tot[1][kSortBins], part_bef[1][kSortBins];
    __shared__ uint32_t base_s[kSortBins], tot_s[kSortBins], half_cnt[2][kSortBins];
    uint32_t* hist_s = dyn_smem;
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const float* __restrict__ losses = p.losses;
    const int64_t N = p.N;
    constexpr int64_t kTileElems = int64_t{kThreads} * E;
    const int64_t tiles_n = (N + kTileElems - 1) / kTileElems;
    StatusBlock* status = p.ws.status;
    uint32_t epoch = 0;

    for (int i = tid; i < kSelBins; i += kThreads) hist_s[i] = 0;
    if (tid < 3) red[tid] = 0;
    grid_dependency_wait();  // the losses (and the scorer's histogram) are complete from here on

    // the block's first tile stays in registers through all phases of the selection
    uint32_t key0[E];
    load_keys<E>(losses, N, static_cast<int64_t>(blockIdx.x) * kTileElems + static_cast<int64_t>(tid) * E, key0);
    // body(tile, keys) for each of this block's tiles: the first from the registers, any further one reloaded
    auto for_each_tile = [&](auto&& body) {
        if (blockIdx.x < tiles_n) body(static_cast<int64_t>(blockIdx.x), key0);
        for (int64_t tile = static_cast<int64_t>(blockIdx.x) + gridDim.x; tile < tiles_n; tile += gridDim.x) {
            uint32_t key[E];
            load_keys<E>(losses, N, tile * kTileElems + static_cast<int64_t>(tid) * E, key);
            body(tile, key);
        }
    };

    // ---- 1. radix select ----
    uint32_t prefix = 0, want = p.k;
    if (p.hist0_ready) {
        uint32_t bin;
        find_bin<true>(p.ws.hist, kSelBins, want, bin, warp_tot, result);
        prefix = bin << 21;
    }
    for (int pass = p.hist0_ready ? 1 : 0; pass < kSelPasses; ++pass) {
        const uint32_t mask = prefix_mask(pass);
        __syncthreads();  // hist_s is zero
        for_each_tile([&](int64_t, const uint32_t (&key)[E]) {
#pragma unroll
            for (int i = 0; i < E; ++i) {
                const bool in = key[i] != 0u && (key[i] & mask) == prefix;
                // plain shared-memory atomics: measured faster than warp-aggregated ones (match.any) for crowded, uniform and
                // all-equal keys alike
                if (in) atomicAdd(&hist_s[digit_of(key[i], pass)], 1u);
            }
        });
        __syncthreads();
        uint32_t* gh = p.ws.hist + pass * kSelBins;
        for (int i = tid; i < kSelBins; i += kThreads) {
            const uint32_t c = hist_s[i];
            if (c) atomicAdd(&gh[i], c);
            hist_s[i] = 0;
        }
        if (!grid_sync(status, epoch, p.barrier_parties, p.barrier_polls)) return;
        uint32_t bin;
        find_bin<true>(gh, pass == 2 ? 1024 : kSelBins, want, bin, warp_tot, result);
        prefix |= pass == 0 ? bin << 21 : pass == 1 ? bin << 10 : bin;
    }
    const uint32_t T = prefix, r = want;  // the k-th key, and how many entries equal to it are selected

    // ---- 2. per tile: keys above T, keys equal to T, largest key ----
    for_each_tile([&](int64_t tile, const uint32_t (&key)[E]) {
        uint32_t gt = 0, eq = 0, mx = 0;
#pragma unroll
        for (int i = 0; i < E; ++i) {
            gt += key[i] > T;
            eq += key[i] == T;
            mx = max(mx, key[i]);
        }
        uint32_t packed = gt | (eq << 16);  // a tile has at most 16,384 entries
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) {
            packed += __shfl_xor_sync(0xFFFFFFFFu, packed, o);
            mx = max(mx, __shfl_xor_sync(0xFFFFFFFFu, mx, o));
        }
        if (lane == 0) {
            atomicAdd(&red[0], packed & 0xFFFFu);
            atomicAdd(&red[1], packed >> 16);
            atomicMax(&red[2], mx);
        }
        __syncthreads();
        if (tid == 0) {
            __stcg(reinterpret_cast<uint4*>(p.ws.tile_counts) + tile, make_uint4(red[0], red[1], red[2], 0u));
            red[0] = red[1] = red[2] = 0;
        }
        __syncthreads();
    });
    if (!grid_sync(status, epoch, p.barrier_parties, p.barrier_polls)) return;

    // ---- 3. ordered compaction ----
    // The sort key of a selected entry is u = kmax - key (0 for the largest loss); `passes` 9-bit digits cover its range.
    uint32_t kmax = 0;
    for (int64_t t = tid; t < tiles_n; t += kThreads) kmax = max(kmax, __ldcg(p.ws.tile_counts + 4 * t + 2));
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) kmax = max(kmax, __shfl_xor_sync(0xFFFFFFFFu, kmax, o));
    if (lane == 0) atomicMax(&red[2], kmax);
    __syncthreads();
    kmax = red[2];
    __syncthreads();
    const uint32_t range = kmax - T;
    const int passes = p.order == LSGD_ORDER_INDEX_ASC ? 0 : (32 - __clz(range) + kSortBits - 1) / kSortBits;
    const bool direct = passes == 0;  // index order is the final order
    const uint32_t tile_entries = 1024u * static_cast<uint32_t>(p.sort_rounds);
    const uint32_t St = p.sort_tiles;
    for_each_tile([&](int64_t tile, const uint32_t (&key)[E]) {
        // entries above / equal to the threshold in the tiles before this one
        if (tid < 2) red[tid] = 0;
        __syncthreads();
        uint32_t gt = 0, eq = 0;
        for (int64_t t = tid; t < tile; t += kThreads) {
            const uint2 c = __ldcg(reinterpret_cast<const uint2*>(p.ws.tile_counts + 4 * t));
            gt += c.x;
            eq += c.y;
        }
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) {
            gt += __shfl_xor_sync(0xFFFFFFFFu, gt, o);
            eq += __shfl_xor_sync(0xFFFFFFFFu, eq, o);
        }
        if (lane == 0 && (gt | eq)) {
            atomicAdd(&red[0], gt);
            atomicAdd(&red[1], eq);
        }
        __syncthreads();
        const uint32_t gt_before = red[0], eq_before = red[1];
        uint32_t my_gt = 0, my_eq = 0;
#pragma unroll
        for (int i = 0; i < E; ++i) {
            my_gt += key[i] > T;
            my_eq += key[i] == T;
        }
        // one scan for both counts: each is at most 16,384 < 2^16
        const uint32_t packed = block_exclusive_scan(my_gt | (my_eq << 16), warp_tot);
        uint32_t gt_run = gt_before + (packed & 0xFFFFu);
        uint32_t eq_run = eq_before + (packed >> 16);
        const int64_t base = tile * kTileElems + static_cast<int64_t>(tid) * E;
#pragma unroll
        for (int i = 0; i < E; ++i) {
            const bool above = key[i] > T;
            const bool tie = key[i] == T;
            if (above || (tie && eq_run < r)) {
                const uint32_t pos = gt_run + min(eq_run, r);
                const int64_t j = base + i;
                if (direct) {
                    p.out_idx[pos] = static_cast<int32_t>(j);
                    if (p.out_vals) p.out_vals[pos] = losses[j];
                } else {
                    __stcg(p.ws.pairs[0] + pos, make_uint2(key[i], static_cast<uint32_t>(j)));
                }
            }
            gt_run += above;
            eq_run += tie;
        }
        __syncthreads();
    });
    if (direct) return;
    if (!grid_sync(status, epoch, p.barrier_parties, p.barrier_polls)) return;

    // ---- 4. stable LSD sort of the k pairs on u = kmax - key, ascending, 9 bits per pass ----
    // A pass has two halves with a barrier between them: every tile ranks its entries by the pass's digit
    // (which also yields the tile's digit counts, written to tile_hist); then every tile reads all tiles' counts,
    // derives where its runs start, and scatters.  A block with a single tile keeps its ranks in registers and
    // shared memory across the barrier; a block with several tiles ranks each of them a second time.
    uint32_t(*counters)[kCounterPitch] = reinterpret_cast<uint32_t(*)[kCounterPitch]>(dyn_smem);
    const int R = p.sort_rounds;
    const uint32_t k = p.k;
    const bool one_tile = St <= gridDim.x;
    uint32_t key[kSortMaxRounds], rank[kSortMaxRounds];
    int32_t idx[kSortMaxRounds];
    for (int pass = 0; pass < passes; ++pass) {
        const bool last = pass == passes - 1;
        const int shift = kSortBits * pass;
        const uint2* pairs_in = p.ws.pairs[pass & 1];
        uint2* pairs_out = p.ws.pairs[(pass + 1) & 1];
        uint32_t* cnt = p.ws.tile_hist;  // [St][kSortBins], rewritten by every pass

        // Loads a tile, ranks its entries stably by this pass's digit: afterwards rank[rd] is the entry's rank
        // among the entries of its warp with the same digit, counters[w][d] the number of such entries in the
        // warps before w of the same half of the block, half_cnt[h][d] the count of half h.
        auto rank_tile = [&](uint32_t tile, bool publish) {
            for (int i = tid; i < kWarps * kCounterPitch; i += kThreads) dyn_smem[i] = 0;
            const uint32_t first = tile * tile_entries + warp * (R * 32);
#pragma unroll
            for (int rd = 0; rd < kSortMaxRounds; ++rd) {  // all loads first: they are independent
                const uint32_t e = first + rd * 32 + lane;
                const bool live = rd < R && e < k;
                const uint2 pr = live ? __ldcg(pairs_in + e) : make_uint2(0u, 0u);
                key[rd] = pr.x;
                idx[rd] = static_cast<int32_t>(pr.y);
            }
            __syncthreads();
#pragma unroll
            for (int rd = 0; rd < kSortMaxRounds; ++rd) {
                if (rd < R) {
                    const uint32_t e = first + rd * 32 + lane;
                    const bool live = e < k;
                    const uint32_t dd = ((kmax - key[rd]) >> shift) & (kSortBins - 1);
                    const uint32_t peers = match_digit(dd, live);
                    const int leader = live ? __ffs(peers) - 1 : lane;
                    uint32_t old = 0;
                    if (live && lane == leader) {
                        old = counters[warp][dd];
                        counters[warp][dd] = old + __popc(peers);
                    }
                    old = __shfl_sync(0xFFFFFFFFu, old, leader);
                    rank[rd] = old + __popc(peers & ((1u << lane) - 1u));
                    __syncwarp();
                }
            }
            __syncthreads();
            {   // per digit, exclusive prefix of the warps' counts within each half of the block: thread (digit, half)
                const int d = tid & (kSortBins - 1), h = tid / kSortBins;
                constexpr int kHalf = kWarps / 2;
                uint32_t c[kHalf];
#pragma unroll
                for (int u = 0; u < kHalf; ++u) c[u] = counters[kHalf * h + u][d];
                uint32_t run = 0;
#pragma unroll
                for (int u = 0; u < kHalf; ++u) {
                    counters[kHalf * h + u][d] = run;
                    run += c[u];
                }
                half_cnt[h][d] = run;
            }
            __syncthreads();
            if (publish && tid < kSortBins) __stcg(cnt + static_cast<size_t>(tile) * kSortBins + tid, half_cnt[0][tid] + half_cnt[1][tid]);
        };

        if (one_tile) {
            if (blockIdx.x < St) rank_tile(blockIdx.x, true);
        } else {
            for (uint32_t tile = blockIdx.x; tile < St; tile += gridDim.x) rank_tile(tile, true);
        }
        if (!grid_sync(status, epoch, p.barrier_parties, p.barrier_polls)) return;

        for (uint32_t tile = blockIdx.x; tile < St; tile += gridDim.x) {
            if (!one_tile) {
                __syncthreads();
                rank_tile(tile, false);
            }
            // where each digit's run starts for this tile: all entries of smaller digits, plus this digit's
            // entries in earlier tiles.  A thread reads four digits' counts of a tile at once (16 bytes; a warp one
            // contiguous 512 bytes) for every eighth tile and adds its sums into shared memory: a quarter of the
            // requests that one 4-byte read per digit and tile took, which is what this step's time went by.
            {
                if (tid < kSortBins) {
                    part_tot[0][tid] = 0;
                    part_bef[0][tid] = 0;
                }
                __syncthreads();
                constexpr int kCols = kSortBins / 4, kTileGroups = kThreads / kCols;
                const int c4 = tid & (kCols - 1), tg = tid / kCols;
                uint4 tot = make_uint4(0u, 0u, 0u, 0u), bef = make_uint4(0u, 0u, 0u, 0u);
                for (uint32_t t0 = tg; t0 < St; t0 += kTileGroups * 8) {
                    uint4 c[8];
#pragma unroll
                    for (int u = 0; u < 8; ++u) {  // eight independent loads in flight
                        const uint32_t t = t0 + u * kTileGroups;
                        c[u] = t < St ? __ldcg(reinterpret_cast<const uint4*>(cnt + static_cast<size_t>(t) * kSortBins) + c4)
                                      : make_uint4(0u, 0u, 0u, 0u);
                    }
#pragma unroll
                    for (int u = 0; u < 8; ++u) {
                        const bool earlier = t0 + u * kTileGroups < tile;
                        tot.x += c[u].x; tot.y += c[u].y; tot.z += c[u].z; tot.w += c[u].w;
                        bef.x += earlier ? c[u].x : 0u; bef.y += earlier ? c[u].y : 0u;
                        bef.z += earlier ? c[u].z : 0u; bef.w += earlier ? c[u].w : 0u;
                    }
                }
                const uint32_t tv[4] = {tot.x, tot.y, tot.z, tot.w}, bv[4] = {bef.x, bef.y, bef.z, bef.w};
#pragma unroll
                for (int e = 0; e < 4; ++e) {  // (sums of counts: the order of the additions does not matter)
                    if (tv[e]) atomicAdd(&part_tot[0][4 * c4 + e], tv[e]);
                    if (bv[e]) atomicAdd(&part_bef[0][4 * c4 + e], bv[e]);
                }
            }
            __syncthreads();
            {
                const bool mine = tid < kSortBins;
                digit_bases(mine ? part_tot[0][tid] : 0u, mine ? part_bef[0][tid] : 0u, tot_s, base_s);
            }
            const uint32_t first = tile * tile_entries + warp * (R * 32);
#pragma unroll
            for (int rd = 0; rd < kSortMaxRounds; ++rd) {
                if (rd < R) {
                    const uint32_t e = first + rd * 32 + lane;
                    if (e < k) {
                        const uint32_t dd = ((kmax - key[rd]) >> shift) & (kSortBins - 1);
                        const uint32_t pos = base_s[dd] + counters[warp][dd] + (warp >= kWarps / 2 ? half_cnt[0][dd] : 0u) + rank[rd];
                        if (last) {
                            p.out_idx[pos] = idx[rd];
                            if (p.out_vals) p.out_vals[pos] = loss_of_key(key[rd], losses, idx[rd]);
                        } else {
                            __stcg(pairs_out + pos, make_uint2(key[rd], static_cast<uint32_t>(idx[rd])));
                        }
                    }
                }
            }
        }
        if (!last && !grid_sync(status, epoch, p.barrier_parties, p.barrier_polls)) return;
    }
}

// ---------------------------------------------------------------------------
// Pools of up to 65,536 entries: ONE thread-block cluster, everything that blocks exchange kept in (distributed)
// shared memory.  Block b owns a slice of 4,096 or 8,192 consecutive entries of the pool (in registers).  Digit
// histograms of the selection are added up in the workspace (global atomics) and every block resolves the digit for
// itself after one barrier.  The barrier is the cluster's hardware barrier.  Two kernels:
//   topk_cluster_kernel         index-ascending output: exact threshold (three digits), per-block counts, ordered
//                               compaction straight into the output;
//   topk_cluster_sorted_kernel  loss-descending output: see there.
// ---------------------------------------------------------------------------
namespace cg = cooperative_groups;

// A 16-byte read from a shared-memory address of another block of the cluster (explicit instructions: reads written
// one after the other are issued one after the other, before the first use).
__device__ __forceinline__ uint4 ld_cluster_v4(uint32_t addr) {
    uint4 v;
    asm volatile("ld.shared::cluster.v4.u32 {%0, %1, %2, %3}, [%4];" : "=r"(v.x), "=r"(v.y), "=r"(v.z), "=r"(v.w) : "r"(addr) : "memory");
    return v;
}

// Digits `first`..`last` (0 = most significant) of the radix selection among the keys a cluster holds in registers.
// hist_s: kSelBins zeroed words of this block (left zeroed); ghist: the workspace's [kSelPasses][kSelBins] histograms,
// those of the digits asked for zeroed.  Every block adds its counts to the global histogram, and after ONE cluster
// barrier every block resolves the digit for itself.  (Adding them into block 0's shared memory instead cost 1.2 to 2.4 us
// a digit for the additions alone, all aimed at one multiprocessor, plus a second barrier to spread the answer.)
// On return `prefix` holds the resolved digits and `want` the rank left inside that prefix.
template <int CE>
__device__ __forceinline__ void cluster_select_digits(cg::cluster_group& cluster, const uint32_t (&key)[CE], int first, int last,
                                                      uint32_t* hist_s, uint32_t* ghist, uint32_t* warp_tot, uint32_t* result,
                                                      uint32_t& prefix, uint32_t& want) {
    const int tid = threadIdx.x;
    for (int pass = first; pass <= last; ++pass) {
        const uint32_t mask = prefix_mask(pass);
        __syncthreads();  // hist_s is zero
#pragma unroll
        for (int i = 0; i < CE; ++i) {
            const bool in = key[i] != 0u && (key[i] & mask) == prefix;
            // plain shared-memory atomics: measured faster than warp-aggregated ones (match.any) for crowded, uniform and
            // all-equal keys alike
            if (in) atomicAdd(&hist_s[digit_of(key[i], pass)], 1u);
        }
        __syncthreads();
        for (int i = tid; i < kSelBins; i += kThreads) {
            const uint32_t c = hist_s[i];
            if (c) atomicAdd(ghist + pass * kSelBins + i, c);
            hist_s[i] = 0;
        }
        cluster.sync();  // every block's additions are in
        uint32_t bin;
        find_bin<true>(ghist + pass * kSelBins, pass == 2 ? 1024 : kSelBins, want, bin, warp_tot, result);
        prefix |= pass == 0 ? bin << 21 : pass == 1 ? bin << 10 : bin;
    }
}

// CE keys per thread (blocks of 1024 CE entries), at most CB blocks: 4 x 16 (a cluster of more than 8 blocks needs the
// device's consent, see launch_topk) or 8 x 8.
template <int CE, int CB>
struct ClusterLayout {
    static constexpr int kTile = kThreads * CE;
    static constexpr size_t kHistBytes = sizeof(uint32_t) * kSelBins;
    static constexpr size_t kSmemBytes = kHistBytes + sizeof(uint4) * CB;
};

template <int CE, int CB>
__global__ void __launch_bounds__(kThreads, 1) topk_cluster_kernel(const __grid_constant__ SelectParams p) {
    using Lay = ClusterLayout<CE, CB>;
    constexpr int kClE = CE, kClTile = Lay::kTile;
    extern __shared__ __align__(16) unsigned char cl_smem[];
    uint32_t* hist_s = reinterpret_cast<uint32_t*>(cl_smem);
    uint4* cta_cnt = reinterpret_cast<uint4*>(cl_smem + Lay::kHistBytes);
    __shared__ uint32_t warp_tot[kWarps + 1];
    __shared__ uint32_t result[3];
    __shared__ uint32_t red[2];
    cg::cluster_group cluster = cg::this_cluster();
    const int tid = threadIdx.x, lane = tid & 31;
    const uint32_t rank = blockIdx.x, nblocks = gridDim.x;
    const float* __restrict__ losses = p.losses;
    const int64_t N = p.N;

    for (int i = tid; i < kSelBins; i += kThreads) hist_s[i] = 0;
    if (tid < 2) red[tid] = 0;
    grid_dependency_wait();  // the losses (and the scorer's histogram) are complete from here on

    if (p.standalone) {
        // a selection on its own: the status block reads "nothing to report", and block 0 clears the workspace's
        // histograms (a fused call's memset has done both)
        if (rank == 0) {
            if (tid == 0) {
                p.ws.status->bad_labels = 0;
                p.ws.status->timeout = 0;
            }
            for (int i = tid; i < kSelPasses * kSelBins; i += kThreads) p.ws.hist[i] = 0;
        }
        cluster.sync();
    }
    uint32_t key[kClE];
    load_keys<kClE>(losses, N, static_cast<int64_t>(rank) * kClTile + static_cast<int64_t>(tid) * kClE, key);

    // ---- 1. radix select: the key T of the k-th entry and r, the entries equal to T that are still selected ----
    uint32_t prefix = 0, want = p.k;
    if (p.hist0_ready) {
        uint32_t bin;
        find_bin<true>(p.ws.hist, kSelBins, want, bin, warp_tot, result);
        prefix = bin << 21;
    }
    cluster_select_digits<kClE>(cluster, key, p.hist0_ready ? 1 : 0, kSelPasses - 1, hist_s, p.ws.hist, warp_tot, result, prefix, want);
    const uint32_t T = prefix, r = want;

    // ---- 2. per block: keys above T, keys equal to T; every block gets every block's ----
    uint32_t my_gt = 0, my_eq = 0;
    {
#pragma unroll
        for (int i = 0; i < kClE; ++i) {
            my_gt += key[i] > T;
            my_eq += key[i] == T;
        }
        uint32_t packed = my_gt | (my_eq << 16);
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) packed += __shfl_xor_sync(0xFFFFFFFFu, packed, o);
        if (lane == 0) {
            atomicAdd(&red[0], packed & 0xFFFFu);
            atomicAdd(&red[1], packed >> 16);
        }
        __syncthreads();
        if (tid < static_cast<int>(nblocks)) cluster.map_shared_rank(cta_cnt, tid)[rank] = make_uint4(red[0], red[1], 0u, 0u);
    }
    cluster.sync();  // the last access to another block's shared memory is before this barrier

    // ---- 3. ordered compaction, straight into the output ----
    uint32_t gt_before = 0, eq_before = 0;
    for (uint32_t b = 0; b < rank; ++b) {
        const uint4 c = cta_cnt[b];
        gt_before += c.x;
        eq_before += c.y;
    }
    const uint32_t packed = block_exclusive_scan(my_gt | (my_eq << 16), warp_tot);
    uint32_t gt_run = gt_before + (packed & 0xFFFFu);
    uint32_t eq_run = eq_before + (packed >> 16);
    const int64_t base = static_cast<int64_t>(rank) * kClTile + static_cast<int64_t>(tid) * kClE;
#pragma unroll
    for (int i = 0; i < kClE; ++i) {
        const bool above = key[i] > T;
        const bool tie = key[i] == T;
        if (above || (tie && eq_run < r)) {
            const uint32_t pos = gt_run + min(eq_run, r);
            const int64_t j = base + i;
            p.out_idx[pos] = static_cast<int32_t>(j);
            if (p.out_vals) p.out_vals[pos] = losses[j];
        }
        gt_run += above;
        eq_run += tie;
    }
}

// Loss-descending output.  The selection stops after two digits: every key that shares the 22 resolved bits with the
// k-th key, or lies above them, is a candidate (k' >= k of them: k plus the few keys in the k-th key's bin of 1,024
// consecutive keys); after one digit already where that leaves at most 2 k candidates that fit the tiles k needs.
// The candidates are sorted whole, stably, by v = key - T (T = the lowest key of that bin) in
// descending 9-bit digits, least significant first; the first k positions of the result are the selection, ties
// between equal keys in index order because the candidates start in index order.  No threshold has to be exact and
// no tie has to be counted before the sort.
//
// One cluster barrier per sort pass.  The digit histograms of ALL passes are taken at once from the registers, so
// where a digit's run starts is known up front; what a pass still needs, how many entries with the same digit sit in
// the tiles before a block's own, is counted one pass ahead: while a block scatters its entries it counts, per
// destination tile, the NEXT digit of what it sends there (flow[t][d]), turns the counts into running sums over t,
// and after the barrier the owner of tile t adds up row t of every block's matrix.  Reading another block's shared
// memory is slow (some 30 KB per microsecond and block, measured), so these counts travel as 16-bit halves (no
// block holds more than 8,192 entries) and every read is issued together with seven others.
// Sort tile b (1,024 R consecutive positions, R = 1, 2, 4 or 8 as k' needs) is block b's pair buffer.  For pass 0 every
// warp first packs the candidates among its 32 CE entries (dealt to its lanes so that rounds run through consecutive
// indices), in order, into a list of its own, which it then treats like a slice of a tile.
template <int CE, int CB>
struct SortedClusterLayout {
    static constexpr int kTile = kThreads * CE;
    static constexpr size_t kCountersBytes = sizeof(uint16_t) * kWarps * kSortBins;  // per-warp digit counters; the selection's hist_s before
    static constexpr size_t kPairsBytes = sizeof(uint2) * 2 * kTile;                 // two (key, index) buffers
    static constexpr size_t kFlowBytes = sizeof(uint16_t) * 2 * CB * kSortBins;      // flow[2][CB][kSortBins]; the second one holds the four digit histograms first
    static constexpr size_t kSmemBytes = kCountersBytes + kPairsBytes + kFlowBytes;
    static_assert(sizeof(uint32_t) * kSelBins <= kCountersBytes, "the selection's block histogram fits in the counters");
    static_assert(4 <= CB, "the digit histograms fit in one flow matrix");
    static_assert(CE <= kSortMaxRounds && kTile <= 8192 && kTile < 65536, "a block's digit counts fit 16 bits");
};

template <int CE, int CB>
__global__ void __launch_bounds__(kThreads, 1) topk_cluster_sorted_kernel(const __grid_constant__ SelectParams p) {
    using Lay = SortedClusterLayout<CE, CB>;
    constexpr int kClTile = Lay::kTile;
    constexpr int kRowWords = kSortBins / 2;      // one row of 16-bit digit counts, in 32-bit words
    constexpr int kFlowWords = CB * kRowWords;
    constexpr int kDigits = 4;  // 9 + 9 + 9 + 5 bits
    extern __shared__ __align__(16) unsigned char cl_smem[];
    uint32_t* hist_s = reinterpret_cast<uint32_t*>(cl_smem);
    uint16_t(*counters)[kSortBins] = reinterpret_cast<uint16_t(*)[kSortBins]>(cl_smem);
    uint2* pairs = reinterpret_cast<uint2*>(cl_smem + Lay::kCountersBytes);
    uint32_t* flow = reinterpret_cast<uint32_t*>(cl_smem + Lay::kCountersBytes + Lay::kPairsBytes);  // [2][CB][kRowWords], two digits a word
    uint32_t* dig_hist = flow + kFlowWords;                                                          // [kDigits][kRowWords]
    __shared__ uint32_t warp_tot[kWarps + 1];
    __shared__ uint32_t result[3];
    __shared__ uint32_t vmax_s, vmax_all_s;
    __shared__ uint32_t warp_sum[kWarps];
    __shared__ uint32_t acc_s[2][kRowWords];  // sums of what is read from the other blocks, two digits a word: all of them; the blocks before this one
    __shared__ __align__(16) uint32_t base_s[kDigits][kSortBins];  // entries whose digit is larger, per pass
    __shared__ __align__(16) uint32_t tilebase_s[kSortBins];       // the same plus the entries of the same digit in the tiles before this one
    __shared__ uint32_t half_cnt[2][kSortBins];
    cg::cluster_group cluster = cg::this_cluster();
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const uint32_t rank = blockIdx.x, nblocks = gridDim.x;
    const float* __restrict__ losses = p.losses;
    const int64_t N = p.N;
    const uint4 zero4 = make_uint4(0u, 0u, 0u, 0u);

    for (int i = tid; i < kSelBins; i += kThreads) hist_s[i] = 0;
    for (int i = tid; i < 2 * kFlowWords / 4; i += kThreads) reinterpret_cast<uint4*>(flow)[i] = zero4;
    if (tid < 2 * kRowWords) acc_s[0][tid] = 0;
    if (tid == 0) vmax_s = 0;
    grid_dependency_wait();  // the losses (and the scorer's histogram) are complete from here on

    // The cluster's digit totals of sort passes 1 to 3 are added up in global memory too, in the workspace's third
    // selection histogram (this kernel resolves two digits only).
    uint32_t* digit_totals = p.ws.hist + 2 * kSelBins;  // [3][kSortBins]
    if (p.standalone) {
        // a selection on its own: the status block reads "nothing to report", and block 0 clears the workspace's
        // histograms (a fused call's memset has done both)
        if (rank == 0) {
            if (tid == 0) {
                p.ws.status->bad_labels = 0;
                p.ws.status->timeout = 0;
            }
            for (int i = tid; i < kSelPasses * kSelBins; i += kThreads) p.ws.hist[i] = 0;
        }
        cluster.sync();
    }
    // entry (round i, lane l) of warp w: index block start + 32 CE w + 32 i + l
    const int64_t wbase = static_cast<int64_t>(rank) * kClTile + static_cast<int64_t>(warp) * (32 * CE) + lane;
    uint32_t key[CE];
#pragma unroll
    for (int i = 0; i < CE; ++i) {
        const int64_t j = wbase + 32 * i;
        key[i] = j < N ? loss_key(losses[j]) : 0u;
    }

    // ---- 1. the leading digit of the k-th key, and the second one unless the first leaves few enough candidates ----
    uint32_t prefix = 0, want = p.k;
    if (p.hist0_ready) {
        uint32_t bin;
        find_bin<true>(p.ws.hist, kSelBins, want, bin, warp_tot, result);
        prefix = bin << 21;
    } else {
        cluster_select_digits<CE>(cluster, key, 0, 0, hist_s, p.ws.hist, warp_tot, result, prefix, want);
    }
    {
        // every key of the first digit's bin and above: if sorting them all needs no larger tiles than the selection
        // itself and at most twice the entries, the second digit's exchange costs more than it saves
        const uint32_t all = p.k - want + result[2];
        uint32_t cap = nblocks * 1024u;
        while (cap < p.k) cap <<= 1;
        if (all > cap || all > 2 * p.k) cluster_select_digits<CE>(cluster, key, 1, 1, hist_s, p.ws.hist, warp_tot, result, prefix, want);
    }
    const uint32_t T = prefix;  // candidates: key >= T (and a real key: padding is 0)

    // ---- 2. this block's digit histograms of v = key - T for all passes, its largest v, and each warp's
    //         candidates packed in index order into the second pair buffer ----
    uint2* stage = pairs + kClTile + warp * (32 * CE);
    uint32_t cnt_w = 0;  // entries this warp ranks in the coming pass
    {
        uint32_t vm = 0;
#pragma unroll
        for (int i = 0; i < CE; ++i) {
            const bool cand = key[i] != 0u && key[i] >= T;
            const uint32_t votes = __ballot_sync(0xFFFFFFFFu, cand);
            if (cand) {
                const uint32_t v = key[i] - T;
                vm = max(vm, v);
                const uint32_t d0 = v & (kSortBins - 1), d1 = (v >> kSortBits) & (kSortBins - 1), d2 = (v >> (2 * kSortBits)) & (kSortBins - 1),
                               d3 = v >> (3 * kSortBits);
                atomicAdd(&dig_hist[d0 >> 1], 1u << ((d0 & 1u) * 16));
                atomicAdd(&dig_hist[kRowWords + (d1 >> 1)], 1u << ((d1 & 1u) * 16));
                atomicAdd(&dig_hist[2 * kRowWords + (d2 >> 1)], 1u << ((d2 & 1u) * 16));
                atomicAdd(&dig_hist[3 * kRowWords + (d3 >> 1)], 1u << ((d3 & 1u) * 16));
                stage[cnt_w + __popc(votes & ((1u << lane) - 1u))] = make_uint2(key[i], static_cast<uint32_t>(wbase + 32 * i));
            }
            cnt_w += __popc(votes);
        }
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) vm = max(vm, __shfl_xor_sync(0xFFFFFFFFu, vm, o));
        if (lane == 0 && vm) atomicMax(&vmax_s, vm);
    }
    __syncthreads();
    if (tid < 3 * kRowWords) {  // passes 1 to 3: this block's counts into the cluster's totals
        const uint32_t w = dig_hist[kRowWords + tid];
        if (w & 0xFFFFu) atomicAdd(&digit_totals[2 * tid], w & 0xFFFFu);
        if (w >> 16) atomicAdd(&digit_totals[2 * tid + 1], w >> 16);
    }
    cluster.sync();

    // ---- 3. all blocks' histograms: where each digit's run starts in every pass (larger digits first), the number
    //         of candidates, the number of passes ----
    uint32_t kc;  // k', the candidates
    {
        // Pass 0 needs every block's histogram (how many candidates with the same digit sit in the blocks before this
        // one): thread (other block u, 16-byte piece) reads one piece and adds it to this block's sums, two digits a word
        // (the other blocks hold fewer than 65,536 entries together: no half carries).  Block u is counted from this
        // block's successor, so that no block is read by all at once.  The totals of the later passes come from global memory.
        const uint32_t g1 = __ldcg(digit_totals + tid), g2 = tid < kSortBins ? __ldcg(digit_totals + kThreads + tid) : 0u;
        {
            const int u = tid >> 6, piece = tid & 63;
            if (u < static_cast<int>(nblocks) - 1) {
                uint32_t b = rank + 1 + u;
                b -= b >= nblocks ? nblocks : 0u;
                uint32_t ra;
                asm volatile("mapa.shared::cluster.u32 %0, %1, %2;" : "=r"(ra) : "r"(static_cast<uint32_t>(__cvta_generic_to_shared(dig_hist + 4 * piece))), "r"(b));
                const uint4 c = ld_cluster_v4(ra);
                const uint32_t w[4] = {c.x, c.y, c.z, c.w};
#pragma unroll
                for (int e = 0; e < 4; ++e) {
                    if (w[e]) {
                        atomicAdd(&acc_s[0][4 * piece + e], w[e]);
                        if (b < rank) atomicAdd(&acc_s[1][4 * piece + e], w[e]);
                    }
                }
            }
        }
        if (warp == kWarps - 1) {  // (never one of the readers above)
            uint32_t m = lane < static_cast<int>(nblocks) ? *cluster.map_shared_rank(&vmax_s, lane) : 0u;
#pragma unroll
            for (int o = 16; o > 0; o >>= 1) m = max(m, __shfl_xor_sync(0xFFFFFFFFu, m, o));
            if (lane == 0) vmax_all_s = m;
        }
        base_s[1 + (tid >> 9)][tid & (kSortBins - 1)] = g1;
        if (tid < kSortBins) base_s[3][tid] = g2;
        for (int i = tid; i < static_cast<int>(Lay::kCountersBytes / 16); i += kThreads) reinterpret_cast<uint4*>(cl_smem)[i] = zero4;
        __syncthreads();
        // thread (pass q, pair j): digits 511 - 2 j and 510 - 2 j; a descending exclusive scan per pass
        const int q = tid >> 8, j = tid & 255, lo = kSortBins - 2 - 2 * j;
        uint32_t g_lo, g_hi, b_lo = 0, b_hi = 0;
        if (q == 0) {
            const uint32_t wo = acc_s[0][lo / 2], wb = acc_s[1][lo / 2], wm = dig_hist[lo / 2];
            acc_s[0][lo / 2] = 0;  // clear again for the next pass's sums
            acc_s[1][lo / 2] = 0;
            g_lo = (wo & 0xFFFFu) + (wm & 0xFFFFu), g_hi = (wo >> 16) + (wm >> 16);
            b_lo = wb & 0xFFFFu, b_hi = wb >> 16;
        } else {
            g_lo = base_s[q][lo], g_hi = base_s[q][lo + 1];
        }
        const uint32_t s2 = g_lo + g_hi;
        uint32_t inc = s2;
#pragma unroll
        for (int o = 1; o < 32; o <<= 1) {
            const uint32_t n = __shfl_up_sync(0xFFFFFFFFu, inc, o);
            if (lane >= o) inc += n;
        }
        if (lane == 31) warp_sum[warp] = inc;
        __syncthreads();
        uint32_t below = 0;  // entries of this pass with larger digits, in the warps before this one
#pragma unroll
        for (int w = 0; w < 8; ++w) below += w < (warp & 7) ? warp_sum[(warp & ~7) + w] : 0u;
        const uint32_t start_hi = below + inc - s2;
        base_s[q][lo + 1] = start_hi;
        base_s[q][lo] = start_hi + g_hi;
        if (q == 0) {
            tilebase_s[lo + 1] = start_hi + b_hi;
            tilebase_s[lo] = start_hi + g_hi + b_lo;
        }
        kc = 0;
#pragma unroll
        for (int w = 0; w < 8; ++w) kc += warp_sum[w];
    }
    const uint32_t vmax = vmax_all_s;
    const int passes = max(1, (32 - __clz(vmax) + kSortBits - 1) / kSortBits);
    int R = 1;
    while (nblocks * 1024u * R < kc) R <<= 1;  // R <= CE: the candidates are no more than the pool
    const int tshift = 10 + (R == 1 ? 0 : R == 2 ? 1 : R == 4 ? 2 : 3);
    const uint32_t tmask = (1u << tshift) - 1u;
    const uint32_t k = p.k;

    // ---- 4. the passes: pass 0 from the warps' packed lists, the others tile b in block b ----
    const uint32_t first = (rank << tshift) + warp * (R * 32);  // position of this warp's first entry in passes 1, 2, ...
    uint32_t* cnt32 = reinterpret_cast<uint32_t*>(cl_smem);     // the counters, two digits a word
    for (int pass = 0; pass < passes; ++pass) {
        const bool last = pass == passes - 1;
        const int shift = kSortBits * pass;
        uint2* pairs_out = pairs + (pass & 1) * kClTile;
        uint32_t* flow_out = flow + (pass & 1) * kFlowWords;
        const uint2* src = stage;
        if (pass > 0) {
            const uint32_t* flow_in = flow + ((pass - 1) & 1) * kFlowWords;
            {
                // row `rank` of every block's matrix: thread (block u, 16-byte piece) reads one piece and adds it to this
                // block's sums (what is summed lies in the tiles before this block's own: fewer than 65,536 entries
                // whenever this tile holds any, so no half carries)
                const int u = tid >> 6, piece = tid & 63;
                if (u < static_cast<int>(nblocks)) {
                    uint32_t b = rank + u;
                    b -= b >= nblocks ? nblocks : 0u;
                    uint32_t ra;
                    asm volatile("mapa.shared::cluster.u32 %0, %1, %2;" : "=r"(ra) : "r"(static_cast<uint32_t>(__cvta_generic_to_shared(flow_in + rank * kRowWords + 4 * piece))), "r"(b));
                    const uint4 c = ld_cluster_v4(ra);
                    const uint32_t w[4] = {c.x, c.y, c.z, c.w};
#pragma unroll
                    for (int e = 0; e < 4; ++e)
                        if (w[e]) atomicAdd(&acc_s[0][4 * piece + e], w[e]);
                }
            }
            for (int i = tid; i < static_cast<int>(Lay::kCountersBytes / 16); i += kThreads) reinterpret_cast<uint4*>(cl_smem)[i] = zero4;
            if (!last)
                for (int i = tid; i < kFlowWords / 4; i += kThreads) reinterpret_cast<uint4*>(flow_out)[i] = zero4;
            src = pairs + ((pass - 1) & 1) * kClTile + warp * (R * 32);
            cnt_w = first < kc ? min(kc - first, static_cast<uint32_t>(R * 32)) : 0u;
        }
        // after its last read of another block's shared memory a block signals the barrier that it waits for before it exits
        if (last) cluster.barrier_arrive();
        uint32_t skey[kSortMaxRounds], srank[kSortMaxRounds];
        int32_t sidx[kSortMaxRounds];
#pragma unroll
        for (int rd = 0; rd < kSortMaxRounds; ++rd) {
            const uint32_t e = rd * 32 + lane;
            const uint2 pr = e < cnt_w ? src[e] : make_uint2(T, 0u);
            skey[rd] = pr.x;
            sidx[rd] = static_cast<int32_t>(pr.y);
        }
        __syncthreads();  // counters are zero (pass 0: and the bases are written)
        if (pass > 0 && tid < kRowWords) {
            const uint32_t w = acc_s[0][tid];
            acc_s[0][tid] = 0;
            tilebase_s[2 * tid] = base_s[pass][2 * tid] + (w & 0xFFFFu);
            tilebase_s[2 * tid + 1] = base_s[pass][2 * tid + 1] + (w >> 16);
        }
        // rank by digit within the warp, in round-then-lane order; the warp's digit counts end up in its counter row
#pragma unroll
        for (int rd = 0; rd < kSortMaxRounds; ++rd) {
            if (rd * 32 < cnt_w) {
                const bool live = rd * 32 + lane < cnt_w;
                const uint32_t dd = ((skey[rd] - T) >> shift) & (kSortBins - 1);
                const uint32_t peers = match_digit(dd, live);
                const int leader = live ? __ffs(peers) - 1 : lane;
                uint32_t old = 0;
                if (live && lane == leader) {
                    old = counters[warp][dd];
                    counters[warp][dd] = static_cast<uint16_t>(old + __popc(peers));
                }
                old = __shfl_sync(0xFFFFFFFFu, old, leader);
                srank[rd] = old + __popc(peers & ((1u << lane) - 1u));
                __syncwarp();
            }
        }
        __syncthreads();
        if (tid < kSortBins) {  // per pair of digits, the exclusive prefix of the warps' counts within each half of the block
            const int dp = tid & (kRowWords - 1), h = tid / kRowWords;
            constexpr int kHalf = kWarps / 2;
            uint32_t c[kHalf];
#pragma unroll
            for (int u = 0; u < kHalf; ++u) c[u] = cnt32[(kHalf * h + u) * kRowWords + dp];
            uint32_t run = 0;
#pragma unroll
            for (int u = 0; u < kHalf; ++u) {
                cnt32[(kHalf * h + u) * kRowWords + dp] = run;
                run += c[u];  // at most 16 x 256 a digit: the halves never carry
            }
            half_cnt[h][2 * dp] = run & 0xFFFFu;
            half_cnt[h][2 * dp + 1] = run >> 16;
        }
        __syncthreads();
#pragma unroll
        for (int rd = 0; rd < kSortMaxRounds; ++rd) {
            if (rd * 32 + lane < cnt_w) {
                const uint32_t v = skey[rd] - T, dd = (v >> shift) & (kSortBins - 1);
                const uint32_t pos = tilebase_s[dd] + counters[warp][dd] + (warp >= kWarps / 2 ? half_cnt[0][dd] : 0u) + srank[rd];
                if (last) {
                    if (pos < k) {
                        p.out_idx[pos] = sidx[rd];
                        if (p.out_vals) p.out_vals[pos] = loss_of_key(skey[rd], losses, sidx[rd]);
                    }
                } else {
                    const uint32_t t = pos >> tshift, dn = (v >> (shift + kSortBits)) & (kSortBins - 1);
                    atomicAdd(&flow_out[t * kRowWords + (dn >> 1)], 1u << ((dn & 1u) * 16));
                    cluster.map_shared_rank(pairs_out, t)[pos & tmask] = make_uint2(skey[rd], static_cast<uint32_t>(sidx[rd]));
                }
            }
        }
        if (!last) {
            __syncthreads();
            if (tid < kRowWords) {  // counts per destination tile -> running sums over the tiles (two digits a word, no carries)
                uint32_t c[CB];
#pragma unroll
                for (int t = 0; t < CB; ++t) c[t] = t < static_cast<int>(nblocks) ? flow_out[t * kRowWords + tid] : 0u;
                uint32_t run = 0;
#pragma unroll
                for (int t = 0; t < CB; ++t) {
                    if (t < static_cast<int>(nblocks)) flow_out[t * kRowWords + tid] = run;
                    run += c[t];
                }
            }
            cluster.sync();
        }
    }
    cluster.barrier_wait();  // no block exits while another may still read its shared memory
}

// Small pools, loss-descending output: every entry finds its own position by counting, position = (entries with a
// larger key) + (entries with the same key and a lower index), and writes itself there if that is below k.  No
// sort and no exchange: each block keeps all N keys in shared memory (4 KB), a thread compares its key with four
// others per shared-memory read (all lanes read the same address), and the few blocks run side by side on
// different multiprocessors (N = 1,024: 8 blocks of 128 threads, about 2,300 instructions per thread, against 55
// compare-exchange steps with 30 block barriers of the bitonic network below).
constexpr int kRankThreads = 128;

__global__ void __launch_bounds__(kRankThreads)
small_rank_kernel(const float* __restrict__ losses, int n, int k, int32_t* __restrict__ out_idx,
                  float* __restrict__ out_vals, StatusBlock* status) {
    __shared__ __align__(16) uint32_t keys[kSmallN];
    grid_dependency_wait();
    if (status && blockIdx.x == 0 && threadIdx.x == 0) {  // a selection on its own: "nothing to report"
        status->bad_labels = 0;
        status->timeout = 0;
    }
    const int n4 = (n + 3) >> 2;
#pragma unroll
    for (int u = 0; u < kSmallN / kRankThreads; ++u) {  // (independent loads, all in flight at once)
        const int j = u * kRankThreads + threadIdx.x;
        if (j < 4 * n4) keys[j] = j < n ? loss_key(losses[j]) : 0u;  // key 0: below every loss
    }
    __syncthreads();
    grid_launch_dependents();
    const uint4* kv = reinterpret_cast<const uint4*>(keys);
    for (int i = blockIdx.x * kRankThreads + threadIdx.x; i < n; i += gridDim.x * kRankThreads) {
        const uint32_t me = keys[i];
        const int ci = i >> 2;
        uint32_t r0 = 0, r1 = 0, r2 = 0, r3 = 0;
#pragma unroll 8
        for (int c = 0; c < ci; ++c) {  // lower indices: equal keys come first
            const uint4 q = kv[c];
            r0 += q.x >= me;
            r1 += q.y >= me;
            r2 += q.z >= me;
            r3 += q.w >= me;
        }
        {
            const uint4 q = kv[ci];
            const int e = i & 3;
            r0 += e > 0 ? q.x >= me : false;
            r1 += e > 1 ? q.y >= me : (e < 1 && q.y > me);
            r2 += e > 2 ? q.z >= me : (e < 2 && q.z > me);
            r3 += e < 3 && q.w > me;
        }
#pragma unroll 8
        for (int c = ci + 1; c < n4; ++c) {  // higher indices: only larger keys come first
            const uint4 q = kv[c];
            r0 += q.x > me;
            r1 += q.y > me;
            r2 += q.z > me;
            r3 += q.w > me;
        }
        const uint32_t pos = (r0 + r1) + (r2 + r3);
        if (pos < static_cast<uint32_t>(k)) {
            out_idx[pos] = i;
            if (out_vals) out_vals[pos] = losses[i];
        }
    }
}

// Small pools, index-ascending output: one CTA sorts all N composite keys (key, ~index), one per thread, with a
// bitonic network; the k-th of them is the cut, and the entries at or above it are written in index order.
constexpr int kSmallThreads = 1024;

__global__ void __launch_bounds__(kSmallThreads)
small_topk_kernel(const float* __restrict__ losses, int n, int k, int32_t* __restrict__ out_idx,
                  float* __restrict__ out_vals, StatusBlock* status) {
    __shared__ unsigned long long ck[kSmallN];
    __shared__ uint32_t warp_tot[kSmallThreads / 32];
    grid_dependency_wait();
    if (status && threadIdx.x == 0) {  // a selection on its own: the status block reads "nothing to report"
        status->bad_labels = 0;
        status->timeout = 0;
    }
    int n2 = 1;
    while (n2 < n) n2 <<= 1;
    for (int i = threadIdx.x; i < n2; i += kSmallThreads)
        ck[i] = i < n ? (static_cast<unsigned long long>(loss_key(losses[i])) << 32) | (0xFFFFFFFFu - static_cast<uint32_t>(i))
                      : 0ull;
    __syncthreads();
    static_assert(kSmallN <= kSmallThreads, "one entry per thread");
    {
        // One entry per thread, in a register: steps with stride < 32 exchange by shuffle, the wider ones through
        // shared memory.  Entry i keeps the larger of the pair if it is the lower index of a descending run (or the
        // upper index of an ascending one).
        const int i = threadIdx.x;
        unsigned long long v = i < n2 ? ck[i] : 0ull;
        for (int size = 2; size <= n2; size <<= 1) {
            const bool desc = (i & size) == 0;
            for (int stride = size >> 1; stride > 0; stride >>= 1) {
                unsigned long long pv;
                if (stride >= 32) {
                    __syncthreads();  // the previous round's reads are done
                    if (i < n2) ck[i] = v;
                    __syncthreads();
                    pv = i < n2 ? ck[i ^ stride] : 0ull;
                } else {
                    pv = __shfl_xor_sync(0xFFFFFFFFu, v, stride);
                }
                const bool take_max = ((i & stride) == 0) == desc;
                v = take_max ? (v > pv ? v : pv) : (v < pv ? v : pv);
            }
        }
        __syncthreads();
        if (i < n2) ck[i] = v;
        __syncthreads();
    }
    grid_launch_dependents();
    // an entry is selected iff its composite key is >= the k-th largest
    const unsigned long long cut = ck[k - 1];
    const int j = threadIdx.x;  // one index per thread
    const bool sel = j < n && ((static_cast<unsigned long long>(loss_key(losses[j])) << 32) | (0xFFFFFFFFu - static_cast<uint32_t>(j))) >= cut;
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    uint32_t inc = sel;
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) {
        const uint32_t v = __shfl_up_sync(0xFFFFFFFFu, inc, o);
        if (lane >= o) inc += v;
    }
    if (lane == 31) warp_tot[warp] = inc;
    __syncthreads();
    uint32_t pos = inc - sel;
    for (int w = 0; w < warp; ++w) pos += warp_tot[w];
    if (sel) {
        out_idx[pos] = j;
        if (out_vals) out_vals[pos] = losses[j];
    }
}

// Opts `kernel` in to `bytes` of dynamic shared memory, once per kernel and device (the call costs host time at
// every launch otherwise).  The kernels share one function type, so the memo is keyed by the function's address.
template <typename K>
cudaError_t allow_dynamic_smem(K kernel, size_t bytes) {
    struct Entry {
        const void* fn;
        int dev;
    };
    static std::mutex mu;
    static std::vector<Entry> done;
    int dev = 0;
    cudaError_t e = cudaGetDevice(&dev);
    if (e != cudaSuccess) return e;
    const void* fn = reinterpret_cast<const void*>(kernel);
    {
        std::lock_guard<std::mutex> lock(mu);
        for (const Entry& d : done)
            if (d.fn == fn && d.dev == dev) return cudaSuccess;
    }
    e = cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, static_cast<int>(bytes));
    if (e != cudaSuccess) return e;
    std::lock_guard<std::mutex> lock(mu);
    done.push_back(Entry{fn, dev});
    return cudaSuccess;
}

template <int E>
cudaError_t launch_select(const SelectParams& p, int grid, cudaStream_t s) {
    auto kernel = topk_select_kernel<E>;
    cudaError_t e = allow_dynamic_smem(kernel, kDynSmemBytes);
    if (e != cudaSuccess) return e;
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3(static_cast<unsigned>(grid));
    cfg.blockDim = dim3(kThreads);
    cfg.dynamicSmemBytes = kDynSmemBytes;
    cfg.stream = s;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeCooperative;  // all blocks resident at once, or the launch is refused
    attr[0].val.cooperative = 1;
    cfg.numAttrs = 1;
    cfg.attrs = attr;
    return cudaLaunchKernelEx(&cfg, kernel, p);
}

// One cluster of `grid` blocks; it may be scheduled while the previous kernel of the stream drains (it waits for
// that kernel's completion before its first global access).
inline cudaLaunchConfig_t cluster_config(int grid, size_t smem, cudaStream_t s, cudaLaunchAttribute (&attr)[2]) {
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3(static_cast<unsigned>(grid));
    cfg.blockDim = dim3(kThreads);
    cfg.dynamicSmemBytes = smem;
    cfg.stream = s;
    attr[0].id = cudaLaunchAttributeClusterDimension;
    attr[0].val.clusterDim.x = static_cast<unsigned>(grid);
    attr[0].val.clusterDim.y = 1;
    attr[0].val.clusterDim.z = 1;
    attr[1].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[1].val.programmaticStreamSerializationAllowed = 1;
    cfg.numAttrs = 2;
    cfg.attrs = attr;
    return cfg;
}

template <int CE, int CB>
cudaError_t launch_cluster(const SelectParams& p, int grid, cudaStream_t s) {
    const bool sorted = p.order != LSGD_ORDER_INDEX_ASC;
    auto kernel = sorted ? topk_cluster_sorted_kernel<CE, CB> : topk_cluster_kernel<CE, CB>;
    const size_t smem = sorted ? SortedClusterLayout<CE, CB>::kSmemBytes : ClusterLayout<CE, CB>::kSmemBytes;
    cudaError_t e = allow_dynamic_smem(kernel, smem);
    if (e != cudaSuccess) return e;
    cudaLaunchAttribute attr[2];
    cudaLaunchConfig_t cfg = cluster_config(grid, smem, s, attr);
    return cudaLaunchKernelEx(&cfg, kernel, p);
}

// Whether this device runs the 16-block cluster variant (clusters of more than 8 blocks are an opt-in, and the device
// must be able to co-schedule 16 blocks of this size in one cluster).  Asked once per device.
bool wide_cluster_ok() {
    static std::mutex mu;
    static int known[64] = {0};  // 0 unknown, 1 yes, 2 no
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess) return false;
    std::lock_guard<std::mutex> lock(mu);
    int& k = known[dev & 63];
    if (k == 0) {
        k = 2;
        auto fits = [](auto kernel, size_t smem) {
            if (allow_dynamic_smem(kernel, smem) != cudaSuccess ||
                cudaFuncSetAttribute(kernel, cudaFuncAttributeNonPortableClusterSizeAllowed, 1) != cudaSuccess)
                return false;
            cudaLaunchAttribute attr[2];
            cudaLaunchConfig_t cfg = cluster_config(16, smem, nullptr, attr);
            int clusters = 0;
            return cudaOccupancyMaxActiveClusters(&clusters, kernel, &cfg) == cudaSuccess && clusters >= 1;
        };
        if (fits(topk_cluster_kernel<4, 16>, ClusterLayout<4, 16>::kSmemBytes) &&
            fits(topk_cluster_sorted_kernel<4, 16>, SortedClusterLayout<4, 16>::kSmemBytes))
            k = 1;
        cudaGetLastError();  // a refusal above is an answer, not an error of the call being made
    }
    return k == 1;
}

// Blocks of topk_select_kernel that can be resident at once on the current device (cached per device).
int resident_blocks() {
    static int cache[64] = {0};
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess) return 1;
    int& c = cache[dev & 63];
    if (c == 0) {
        auto kernel = topk_select_kernel<16>;
        int per_sm = 0;
        if (cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, static_cast<int>(kDynSmemBytes)) != cudaSuccess ||
            cudaOccupancyMaxActiveBlocksPerMultiprocessor(&per_sm, kernel, kThreads, kDynSmemBytes) != cudaSuccess || per_sm < 1)
            per_sm = 1;
        c = sm_count() * per_sm;
    }
    return c;
}

}  // namespace

cudaError_t launch_topk(const float* losses, int64_t N, int64_t k, lsgd_order order, int32_t* out_idx,
                        float* out_vals, const TopkWorkspace& ws, bool hist0_ready, bool standalone, cudaStream_t s) {
    if (N <= kSmallN) {
        if (order == LSGD_ORDER_LOSS_DESC) {
            const int grid = static_cast<int>(std::min<int64_t>((N + kRankThreads - 1) / kRankThreads, test_geometry().max_ctas));
            return launch_dependent(small_rank_kernel, grid, kRankThreads, s, losses, static_cast<int>(N), static_cast<int>(k),
                                    out_idx, out_vals, standalone ? ws.status : nullptr);
        }
        return launch_dependent(small_topk_kernel, 1, kSmallThreads, s, losses, static_cast<int>(N), static_cast<int>(k),
                                out_idx, out_vals, standalone ? ws.status : nullptr);
    }
    SelectParams p;
    p.losses = losses;
    p.N = N;
    p.k = static_cast<uint32_t>(k);
    p.order = static_cast<int>(order);
    p.out_idx = out_idx;
    p.out_vals = out_vals;
    p.ws = ws;
    p.hist0_ready = hist0_ready ? 1 : 0;
    p.standalone = standalone ? 1 : 0;
    p.barrier_parties = 0;
    p.barrier_polls = kMaxPolls;
    const TestGeometry tg = test_geometry();
    // One cluster when the pool fits (and the test hook leaves it its blocks): up to 16 blocks of 4,096 entries
    // where the device takes clusters that wide, else up to 8 blocks of 8,192.
    if (!tg.no_cluster && N <= int64_t{kMaxClusterBlocks} * 8192) {
        const int64_t blocks4 = (N + 4095) / 4096, blocks8 = (N + 8191) / 8192;
        const bool wide = blocks4 <= tg.max_ctas && !tg.narrow_cluster && (blocks4 <= 8 || wide_cluster_ok());
        const int grid = static_cast<int>(wide ? blocks4 : blocks8);
        if (grid <= tg.max_ctas) {
            p.sort_rounds = sort_rounds_for(k, grid);
            p.sort_tiles = static_cast<uint32_t>((k + 1024 * p.sort_rounds - 1) / (1024 * p.sort_rounds));
            return wide ? launch_cluster<4, 16>(p, grid, s) : launch_cluster<8, 8>(p, grid, s);
        }
    }
    // the cooperative kernel accumulates histograms in the workspace and counts barrier arrivals in the status block
    if (standalone) {
        const cudaError_t ze = zero_topk_workspace(ws.status, k, s);
        if (ze != cudaSuccess) return ze;
    }
    const int resident = std::max(1, std::min(resident_blocks(), tg.max_ctas));
    p.sort_rounds = sort_rounds_any(k, std::min(resident, kSortDirectTiles));
    p.sort_tiles = static_cast<uint32_t>((k + 1024 * p.sort_rounds - 1) / (1024 * p.sort_rounds));
    auto tiles = [&](int e) { return (N + int64_t{kThreads} * e - 1) / (int64_t{kThreads} * e); };
    const int e = tiles(4) <= resident ? 4 : tiles(8) <= resident ? 8 : tiles(12) <= resident ? 12 : 16;
    const int grid = static_cast<int>(std::min<int64_t>(resident, std::max<int64_t>(tiles(e), p.sort_tiles)));
    p.barrier_parties = static_cast<uint32_t>(grid) + (tg.phantom_block ? 1u : 0u);
    p.barrier_polls = tg.phantom_block ? 1u << 14 : kMaxPolls;
    if (e == 4) return launch_select<4>(p, grid, s);
    if (e == 8) return launch_select<8>(p, grid, s);
    if (e == 12) return launch_select<12>(p, grid, s);
    return launch_select<16>(p, grid, s);
}

}  // namespace lsgd
