// Deterministic loss-based top-k selection (Section 4.2, "Data Allocation for
// Fast Workers": the highest-loss samples go to the fast workers).
//
// Total order: higher loss first, then lower index.  Losses are mapped to
// order-preserving 32-bit keys (loss_key), so everything below is integer work
// and the result is exact and bit-reproducible.
//
// One kernel does the whole selection, in phases separated by a barrier over all
// its thread blocks:
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
// Pools of up to 65,536 entries run as ONE thread-block cluster that keeps all it
// exchanges in distributed shared memory (topk_cluster_kernel: the barrier is the
// cluster's hardware barrier); larger pools as a cooperative launch with one
// block per multiprocessor that exchanges through the workspace (all blocks
// resident by construction; the barrier is an arrival counter in the status
// block, polled with a limit: if it ever ran out, the block would set the status
// block's timeout word and return, and the other blocks would follow).
// Pools of at most kSmallN entries are sorted whole by a single block instead.
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

cudaError_t zero_topk_workspace(void* ws, int64_t k, cudaStream_t s) {
    return cudaMemsetAsync(ws, 0, topk_zero_bytes(k), s);
}

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
        while (ld_acquire(&st->grid_arrivals) < target) {
            if (++polls > max_polls || ((polls & 63u) == 0 && *reinterpret_cast<volatile int32_t*>(&st->timeout) != 0)) {
                ok = 0;
                break;
            }
            __nanosleep(32);
        }
        if (!ok) atomicExch(&st->timeout, 1);
        __threadfence();
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

// Walks a finished histogram (global memory) from its highest bin down and finds the bin that holds the `want`-th
// entry (1-based).  On return (all threads): bin, and `want` reduced by the entries in the bins above it.
template <bool GLOBAL = true>
__device__ void find_bin(const uint32_t* hist, int nbins, uint32_t& want, uint32_t& bin, uint32_t* warp_tot, uint32_t* result) {
    // thread t owns bins nbins - 1 - 2 t and nbins - 2 - 2 t (or the single bin nbins - 1 - t), highest first
    const bool two = nbins == 2 * kThreads;
    const int b0 = two ? nbins - 1 - 2 * static_cast<int>(threadIdx.x) : nbins - 1 - static_cast<int>(threadIdx.x);
    const uint32_t c0 = GLOBAL ? __ldcg(hist + b0) : hist[b0];
    const uint32_t c1 = !two ? 0u : GLOBAL ? __ldcg(hist + b0 - 1) : hist[b0 - 1];
    const uint32_t before = block_exclusive_scan(c0 + c1, warp_tot);
    if (before < want && want <= before + c0 + c1) {
        const bool first = want <= before + c0;
        result[0] = first ? b0 : b0 - 1;
        result[1] = first ? want - before : want - before - c0;
    }
    __syncthreads();
    bin = result[0];
    want = result[1];
    __syncthreads();
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

// E: keys per thread of a selection tile (tiles of 1024 E entries; block b takes tiles b, b + gridDim.x, ...).
template <int E>
__global__ void __launch_bounds__(kThreads, 1) topk_select_kernel(const __grid_constant__ SelectParams p) {
    extern __shared__ __align__(16) uint32_t dyn_smem[];  // selection: hist_s[kSelBins]; sort: counters[kWarps][kCounterPitch]
    __shared__ uint32_t warp_tot[kWarps + 1];
    __shared__ uint32_t result[2];
    __shared__ uint32_t red[3];
    __shared__ uint32_t part_tot[2][kSortBins], part_bef[2][kSortBins];
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
        find_bin(p.ws.hist, kSelBins, want, bin, warp_tot, result);
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
        find_bin(gh, pass == 2 ? 1024 : kSelBins, want, bin, warp_tot, result);
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
    const int tshift = 10 + (p.sort_rounds == 1 ? 0 : p.sort_rounds == 2 ? 1 : p.sort_rounds == 4 ? 2 : 3);
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
            const uint32_t first = (tile << tshift) + warp * (R * 32);
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
            // entries in earlier tiles (two threads per digit, each over half of the tiles)
            {
                const int d = tid & (kSortBins - 1), q = tid / kSortBins;
                const uint32_t per = (St + 1) / 2;
                const uint32_t t_lo = q * per, t_hi = min(St, t_lo + per);
                uint32_t total = 0, bef = 0;
                for (uint32_t t0 = t_lo; t0 < t_hi; t0 += 16) {
                    uint32_t c[16];
#pragma unroll
                    for (int u = 0; u < 16; ++u)  // sixteen independent loads in flight
                        c[u] = t0 + u < t_hi ? __ldcg(cnt + static_cast<size_t>(t0 + u) * kSortBins + d) : 0u;
#pragma unroll
                    for (int u = 0; u < 16; ++u) {
                        total += c[u];
                        bef += t0 + u < tile ? c[u] : 0u;
                    }
                }
                part_tot[q][d] = total;
                part_bef[q][d] = bef;
            }
            __syncthreads();
            {
                const bool mine = tid < kSortBins;
                digit_bases(mine ? part_tot[0][tid] + part_tot[1][tid] : 0u, mine ? part_bef[0][tid] + part_bef[1][tid] : 0u, tot_s, base_s);
            }
            const uint32_t first = (tile << tshift) + warp * (R * 32);
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
// Pools of up to 65,536 entries: the same algorithm as ONE thread-block cluster, everything that blocks exchange
// kept in (distributed) shared memory.  Block b owns a slice of 4,096 or 8,192 consecutive entries of the pool (in
// registers) and sort tile b.  Digit histograms are added into block 0's shared memory and read from
// there by every block; per-block counts, the sort's digit counts and the (key, index) pairs themselves are
// written straight into the destination block's shared memory.  The barrier is the cluster's hardware barrier.
// ---------------------------------------------------------------------------
namespace cg = cooperative_groups;

// CE keys per thread (blocks of 1024 CE entries), at most CB blocks: 4 x 16 (a cluster of more than 8 blocks needs the
// device's consent, see launch_topk) or 8 x 8.
template <int CE, int CB>
struct ClusterLayout {
    static constexpr int kTile = kThreads * CE;
    static constexpr size_t kCountersBytes = sizeof(uint32_t) * kWarps * kCounterPitch;
    static constexpr size_t kPairsBytes = sizeof(uint2) * 2 * kTile;
    static constexpr size_t kMatBytes = sizeof(uint32_t) * CB * kSortBins;
    static constexpr size_t kSmemBytes = kCountersBytes + kPairsBytes + kMatBytes + sizeof(uint4) * CB;
    static_assert(kCountersBytes % 16 == 0, "the pair buffers start 16-byte aligned");
    static_assert(sizeof(uint32_t) * kSelPasses * kSelBins <= kPairsBytes / 2, "the selection's histograms fit in the first pair buffer");
    static_assert(kTile <= 1024 * kSortMaxRounds, "a block's pairs are one sort tile");
};

template <int CE, int CB>
__global__ void __launch_bounds__(kThreads, 1) topk_cluster_kernel(const __grid_constant__ SelectParams p) {
    using Lay = ClusterLayout<CE, CB>;
    constexpr int kClE = CE, kClTile = Lay::kTile;
    extern __shared__ __align__(16) unsigned char cl_smem[];
    uint32_t* dyn = reinterpret_cast<uint32_t*>(cl_smem);                                          // hist_s, later counters
    uint2* pairs = reinterpret_cast<uint2*>(cl_smem + Lay::kCountersBytes);                         // [2][kClTile]
    uint32_t* acc_hist = reinterpret_cast<uint32_t*>(pairs);                                        // block 0, selection only: [3][kSelBins]
    uint32_t* mat = reinterpret_cast<uint32_t*>(cl_smem + Lay::kCountersBytes + Lay::kPairsBytes);   // [blocks][kSortBins]
    uint4* cta_cnt = reinterpret_cast<uint4*>(cl_smem + Lay::kCountersBytes + Lay::kPairsBytes + Lay::kMatBytes);
    __shared__ uint32_t warp_tot[kWarps + 1];
    __shared__ uint32_t result[2];
    __shared__ uint32_t red[3];
    __shared__ uint32_t digit_s[2];  // (bin, rank left) of the digit block 0 resolved last
    __shared__ uint32_t base_s[kSortBins], tot_s[kSortBins], half_cnt[2][kSortBins];
    cg::cluster_group cluster = cg::this_cluster();
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const uint32_t rank = blockIdx.x, nblocks = gridDim.x;
    const float* __restrict__ losses = p.losses;
    const int64_t N = p.N;
    uint32_t* hist_s = dyn;

    for (int i = tid; i < kSelBins; i += kThreads) hist_s[i] = 0;
    for (int i = tid; i < kSelPasses * kSelBins; i += kThreads) acc_hist[i] = 0;
    for (int i = tid; i < CB * kSortBins; i += kThreads) mat[i] = 0;
    if (tid < 3) red[tid] = 0;
    cluster.sync();          // every block's accumulators are clear before anybody adds to them
    grid_dependency_wait();  // the losses (and the scorer's histogram) are complete from here on

    if (p.standalone && rank == 0 && tid == 0) {  // a selection on its own: the status block reads "nothing to report"
        p.ws.status->bad_labels = 0;
        p.ws.status->timeout = 0;
    }
    uint32_t key[kClE];
    load_keys<kClE>(losses, N, static_cast<int64_t>(rank) * kClTile + static_cast<int64_t>(tid) * kClE, key);

    // ---- 1. radix select ----
    uint32_t prefix = 0, want = p.k;
    if (p.hist0_ready) {
        uint32_t bin;
        find_bin(p.ws.hist, kSelBins, want, bin, warp_tot, result);
        prefix = bin << 21;
    }
    for (int pass = p.hist0_ready ? 1 : 0; pass < kSelPasses; ++pass) {
        const uint32_t mask = prefix_mask(pass);
        __syncthreads();  // hist_s is zero
#pragma unroll
        for (int i = 0; i < kClE; ++i) {
            const bool in = key[i] != 0u && (key[i] & mask) == prefix;
            // plain shared-memory atomics: measured faster than warp-aggregated ones (match.any) for crowded, uniform and
            // all-equal keys alike
            if (in) atomicAdd(&hist_s[digit_of(key[i], pass)], 1u);
        }
        __syncthreads();
        uint32_t* acc0 = cluster.map_shared_rank(acc_hist, 0) + pass * kSelBins;
        for (int i = tid; i < kSelBins; i += kThreads) {
            const uint32_t c = hist_s[i];
            if (c) atomicAdd(acc0 + i, c);
            hist_s[i] = 0;
        }
        cluster.sync();
        // block 0 resolves the digit from its own shared memory and tells every block (reading 2,048 bins of
        // another block's shared memory from every block took longer than this second barrier)
        if (rank == 0) {
            uint32_t bin;
            find_bin<false>(acc_hist + pass * kSelBins, pass == 2 ? 1024 : kSelBins, want, bin, warp_tot, result);
            if (tid < static_cast<int>(nblocks)) {
                uint32_t* dst = cluster.map_shared_rank(digit_s, tid);
                dst[0] = bin;
                dst[1] = want;
            }
        }
        cluster.sync();
        const uint32_t bin = digit_s[0];
        want = digit_s[1];
        prefix |= pass == 0 ? bin << 21 : pass == 1 ? bin << 10 : bin;
    }
    const uint32_t T = prefix, r = want;

    // ---- 2. per block: keys above T, keys equal to T, largest key; every block gets every block's ----
    uint32_t my_gt = 0, my_eq = 0;
    {
        uint32_t mx = 0;
#pragma unroll
        for (int i = 0; i < kClE; ++i) {
            my_gt += key[i] > T;
            my_eq += key[i] == T;
            mx = max(mx, key[i]);
        }
        uint32_t packed = my_gt | (my_eq << 16);
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
        if (tid < static_cast<int>(nblocks)) cluster.map_shared_rank(cta_cnt, tid)[rank] = make_uint4(red[0], red[1], red[2], 0u);
    }
    cluster.sync();

    // ---- 3. ordered compaction ----
    uint32_t gt_before = 0, eq_before = 0, kmax = 0;
    for (uint32_t b = 0; b < nblocks; ++b) {
        const uint4 c = cta_cnt[b];
        gt_before += b < rank ? c.x : 0u;
        eq_before += b < rank ? c.y : 0u;
        kmax = max(kmax, c.z);
    }
    const uint32_t range = kmax - T;
    const int passes = p.order == LSGD_ORDER_INDEX_ASC ? 0 : (32 - __clz(range) + kSortBits - 1) / kSortBits;
    const bool direct = passes == 0;
    const int R = p.sort_rounds;
    const int tshift = 10 + (R == 1 ? 0 : R == 2 ? 1 : R == 4 ? 2 : 3);
    const uint32_t tmask = (1u << tshift) - 1u;
    const uint32_t St = p.sort_tiles;  // <= nblocks: sort tile b lives in block b
    {
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
                if (direct) {
                    p.out_idx[pos] = static_cast<int32_t>(j);
                    if (p.out_vals) p.out_vals[pos] = losses[j];
                } else {
                    cluster.map_shared_rank(pairs, pos >> tshift)[pos & tmask] = make_uint2(key[i], static_cast<uint32_t>(j));
                }
            }
            gt_run += above;
            eq_run += tie;
        }
    }
    if (direct) return;  // nobody touches another block's shared memory after the barrier above
    cluster.sync();

    // ---- 4. stable LSD sort on u = kmax - key, 9 bits per pass; tile b = block b's pair buffer ----
    uint32_t(*counters)[kCounterPitch] = reinterpret_cast<uint32_t(*)[kCounterPitch]>(dyn);
    const uint32_t k = p.k;
    const bool has_tile = rank < St;
    const uint32_t first = (rank << tshift) + warp * (R * 32);  // global position of this warp's first entry
    for (int pass = 0; pass < passes; ++pass) {
        const bool last = pass == passes - 1;
        const int shift = kSortBits * pass;
        const uint2* pairs_in = pairs + (pass & 1) * kClTile;
        uint2* pairs_out = pairs + ((pass + 1) & 1) * kClTile;
        uint32_t skey[kSortMaxRounds], srank[kSortMaxRounds];
        int32_t sidx[kSortMaxRounds];
        if (has_tile) {
            for (int i = tid; i < kWarps * kCounterPitch; i += kThreads) dyn[i] = 0;
#pragma unroll
            for (int rd = 0; rd < kSortMaxRounds; ++rd) {
                const uint32_t e = first + rd * 32 + lane;
                const bool live = rd < R && e < k;
                const uint2 pr = live ? pairs_in[e & tmask] : make_uint2(0u, 0u);
                skey[rd] = pr.x;
                sidx[rd] = static_cast<int32_t>(pr.y);
            }
            __syncthreads();
#pragma unroll
            for (int rd = 0; rd < kSortMaxRounds; ++rd) {
                if (rd < R) {
                    const uint32_t e = first + rd * 32 + lane;
                    const bool live = e < k;
                    const uint32_t dd = ((kmax - skey[rd]) >> shift) & (kSortBins - 1);
                    const uint32_t peers = match_digit(dd, live);
                    const int leader = live ? __ffs(peers) - 1 : lane;
                    uint32_t old = 0;
                    if (live && lane == leader) {
                        old = counters[warp][dd];
                        counters[warp][dd] = old + __popc(peers);
                    }
                    old = __shfl_sync(0xFFFFFFFFu, old, leader);
                    srank[rd] = old + __popc(peers & ((1u << lane) - 1u));
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
            // this tile's digit counts, into every block's copy of the count matrix
            for (uint32_t i = tid; i < nblocks * kSortBins; i += kThreads) {
                const uint32_t b = i / kSortBins, d = i % kSortBins;
                cluster.map_shared_rank(mat, b)[rank * kSortBins + d] = half_cnt[0][d] + half_cnt[1][d];
            }
        }
        cluster.sync();
        if (has_tile) {
            {
                uint32_t total = 0, before = 0;
                if (tid < kSortBins) {
                    for (uint32_t b = 0; b < St; ++b) {
                        const uint32_t c = mat[b * kSortBins + tid];
                        total += c;
                        before += b < rank ? c : 0u;
                    }
                }
                digit_bases(total, before, tot_s, base_s);
            }
#pragma unroll
            for (int rd = 0; rd < kSortMaxRounds; ++rd) {
                if (rd < R) {
                    const uint32_t e = first + rd * 32 + lane;
                    if (e < k) {
                        const uint32_t dd = ((kmax - skey[rd]) >> shift) & (kSortBins - 1);
                        const uint32_t pos = base_s[dd] + counters[warp][dd] + (warp >= kWarps / 2 ? half_cnt[0][dd] : 0u) + srank[rd];
                        if (last) {
                            p.out_idx[pos] = sidx[rd];
                            if (p.out_vals) p.out_vals[pos] = loss_of_key(skey[rd], losses, sidx[rd]);
                        } else {
                            cluster.map_shared_rank(pairs_out, pos >> tshift)[pos & tmask] = make_uint2(skey[rd], static_cast<uint32_t>(sidx[rd]));
                        }
                    }
                }
            }
        }
        if (!last) cluster.sync();  // after the last pass's exchange nobody touches another block's shared memory
    }
}

// Small pools: one CTA sorts all N composite keys (key, ~index), one per thread, with a
// bitonic network; the first k are the selection in loss-descending order.
constexpr int kSmallThreads = 1024;

__global__ void __launch_bounds__(kSmallThreads)
small_topk_kernel(const float* __restrict__ losses, int n, int k, int order, int32_t* __restrict__ out_idx,
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
    if (order == LSGD_ORDER_LOSS_DESC) {
        for (int j = threadIdx.x; j < k; j += kSmallThreads) {
            const int32_t i = static_cast<int32_t>(0xFFFFFFFFu - static_cast<uint32_t>(ck[j]));
            out_idx[j] = i;
            if (out_vals) out_vals[j] = losses[i];
        }
        return;
    }
    // index-ascending: an entry is selected iff its composite key is >= the k-th largest
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
template <int CE, int CB>
cudaLaunchConfig_t cluster_config(int grid, cudaStream_t s, cudaLaunchAttribute (&attr)[2]) {
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3(static_cast<unsigned>(grid));
    cfg.blockDim = dim3(kThreads);
    cfg.dynamicSmemBytes = ClusterLayout<CE, CB>::kSmemBytes;
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
    cudaError_t e = allow_dynamic_smem(topk_cluster_kernel<CE, CB>, ClusterLayout<CE, CB>::kSmemBytes);
    if (e != cudaSuccess) return e;
    cudaLaunchAttribute attr[2];
    cudaLaunchConfig_t cfg = cluster_config<CE, CB>(grid, s, attr);
    return cudaLaunchKernelEx(&cfg, topk_cluster_kernel<CE, CB>, p);
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
        auto kernel = topk_cluster_kernel<4, 16>;
        if (allow_dynamic_smem(kernel, ClusterLayout<4, 16>::kSmemBytes) == cudaSuccess &&
            cudaFuncSetAttribute(kernel, cudaFuncAttributeNonPortableClusterSizeAllowed, 1) == cudaSuccess) {
            cudaLaunchAttribute attr[2];
            cudaLaunchConfig_t cfg = cluster_config<4, 16>(16, nullptr, attr);
            int clusters = 0;
            if (cudaOccupancyMaxActiveClusters(&clusters, kernel, &cfg) == cudaSuccess && clusters >= 1) k = 1;
        }
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
    if (N <= kSmallN)
        return launch_dependent(small_topk_kernel, 1, kSmallThreads, s, losses, static_cast<int>(N), static_cast<int>(k),
                                static_cast<int>(order), out_idx, out_vals, standalone ? ws.status : nullptr);
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
    p.sort_rounds = sort_rounds_for(k, std::min(resident, kSortDirectTiles));
    p.sort_tiles = static_cast<uint32_t>((k + 1024 * p.sort_rounds - 1) / (1024 * p.sort_rounds));
    auto tiles = [&](int e) { return (N + int64_t{kThreads} * e - 1) / (int64_t{kThreads} * e); };
    const int e = tiles(4) <= resident ? 4 : tiles(8) <= resident ? 8 : 16;
    const int grid = static_cast<int>(std::min<int64_t>(resident, std::max<int64_t>(tiles(e), p.sort_tiles)));
    p.barrier_parties = static_cast<uint32_t>(grid) + (tg.phantom_block ? 1u : 0u);
    p.barrier_polls = tg.phantom_block ? 1u << 14 : kMaxPolls;
    if (e == 4) return launch_select<4>(p, grid, s);
    if (e == 8) return launch_select<8>(p, grid, s);
    return launch_select<16>(p, grid, s);
}

}  // namespace lsgd
