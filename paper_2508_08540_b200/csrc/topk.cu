// Deterministic loss-based top-k selection (Section 4.2, "Data Allocation for
// Fast Workers": the highest-loss samples go to the fast workers).
//
// Total order: higher loss first, then lower index.  Losses are mapped to
// order-preserving 32-bit keys (loss_key), so everything below is integer work
// and the result is exact and bit-reproducible.
//
//   1. radix select: three histogram passes (11 + 11 + 10 bits, most significant
//      digit first) find the key T of the k-th entry and r, the number of entries
//      equal to T that still belong to the selection;
//   2. ordered compaction: per-tile counts, then an emit pass that keeps every
//      key > T and the r lowest-index keys == T, writing them in index order
//      (scan-based positions: no atomics decide an order);
//   3. for loss-descending output, a stable LSD radix sort (four 8-bit digits) of
//      the k (key, index) pairs; stability turns the index-ascending input order
//      into the required tie-break.  Each scatter pass accumulates the digit
//      counts of the next pass, so the sort is one kernel per digit.
// Pools of at most kSmallN entries are sorted whole by a single CTA instead.
//
// The kernels are short and depend on one another, so their latency is what
// counts: each digit of the threshold is resolved once, by the last CTA to
// finish its histogram pass (a ticket, no waiting), and every kernel is launched
// so that it can be scheduled while its predecessor drains (it waits for the
// predecessor's completion before its first global access).
#include <algorithm>

#include "lsgd_internal.cuh"

namespace lsgd {

// The sort of the selected pairs works on tiles of 1024 entries when k is small (more, shorter CTAs: the pass is
// latency-bound) and of kTile entries otherwise (fewer tiles to prefix over).
constexpr int64_t kSmallSortK = 131072;
static int sort_tile_shift(int64_t k) { return k <= kSmallSortK ? 10 : 12; }
static size_t sort_tiles(int64_t k) { return static_cast<size_t>((k + (int64_t{1} << sort_tile_shift(k)) - 1) >> sort_tile_shift(k)); }
// Tiles reserved for the digit counts: an upper bound of sort_tiles() that grows with k, so that a workspace sized
// for k also serves every smaller k.
static size_t sort_tiles_bound(int64_t k) {
    const size_t small = static_cast<size_t>((std::min<int64_t>(k, kSmallSortK) + 1023) / 1024);
    return std::max(small, static_cast<size_t>((k + kTile - 1) / kTile));
}

size_t topk_workspace_bytes(int64_t N, int64_t k) {
    if (N < 0 || k < 0 || k > N) return 0;
    const size_t tiles_n = static_cast<size_t>((N + kTile - 1) / kTile);
    size_t b = sizeof(StatusBlock);
    b += align_up(sizeof(uint32_t) * kSelPasses * kSelBins);
    b += align_up(sizeof(uint32_t) * 4 * sort_tiles_bound(k) * kSortBins);
    b += align_up(sizeof(uint32_t) * 2 * tiles_n);
    b += 4 * align_up(sizeof(uint32_t) * static_cast<size_t>(k));
    return b;
}

// Bytes at the start of the workspace that one memset must clear before a call.
static size_t topk_zero_bytes(int64_t k) {
    return sizeof(StatusBlock) + align_up(sizeof(uint32_t) * kSelPasses * kSelBins) +
           align_up(sizeof(uint32_t) * 4 * sort_tiles_bound(k) * kSortBins);
}

TopkWorkspace carve_topk(void* ws, int64_t N, int64_t k) {
    const size_t tiles_n = static_cast<size_t>((N + kTile - 1) / kTile);
    unsigned char* p = static_cast<unsigned char*>(ws);
    TopkWorkspace w;
    w.status = reinterpret_cast<StatusBlock*>(p);
    p += sizeof(StatusBlock);
    w.hist = reinterpret_cast<uint32_t*>(p);
    p += align_up(sizeof(uint32_t) * kSelPasses * kSelBins);
    w.tile_hist = reinterpret_cast<uint32_t*>(p);
    p += align_up(sizeof(uint32_t) * 4 * sort_tiles_bound(k) * kSortBins);
    w.tile_counts = reinterpret_cast<uint32_t*>(p);
    p += align_up(sizeof(uint32_t) * 2 * tiles_n);
    const size_t kb = align_up(sizeof(uint32_t) * static_cast<size_t>(k));
    w.keys[0] = reinterpret_cast<uint32_t*>(p);
    w.keys[1] = reinterpret_cast<uint32_t*>(p + kb);
    w.idx[0] = reinterpret_cast<int32_t*>(p + 2 * kb);
    w.idx[1] = reinterpret_cast<int32_t*>(p + 3 * kb);
    return w;
}

cudaError_t zero_topk_workspace(void* ws, int64_t k, cudaStream_t s) {
    return cudaMemsetAsync(ws, 0, topk_zero_bytes(k), s);
}

namespace {

constexpr int kThreads = 256;
constexpr int kPerThread = kTile / kThreads;  // 16

__device__ __forceinline__ uint32_t digit_of(uint32_t key, int pass) {
    return pass == 0 ? key >> 21 : pass == 1 ? (key >> 10) & 0x7FFu : key & 0x3FFu;
}

// Block-wide exclusive scan of one value per thread (kThreads threads).
// `scratch` holds kThreads / 32 + 1 words.  Returns the exclusive prefix; the
// block total is left in scratch[kThreads / 32].
__device__ __forceinline__ uint32_t block_exclusive_scan(uint32_t v, uint32_t* scratch) {
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    uint32_t inc = v;
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) {
        const uint32_t n = __shfl_up_sync(0xFFFFFFFFu, inc, o);
        if (lane >= o) inc += n;
    }
    __syncthreads();  // scratch may still be read from an earlier call
    if (lane == 31) scratch[warp] = inc;
    __syncthreads();
    if (threadIdx.x == 0) {
        uint32_t run = 0;
        for (int w = 0; w < kThreads / 32; ++w) {
            const uint32_t c = scratch[w];
            scratch[w] = run;
            run += c;
        }
        scratch[kThreads / 32] = run;
    }
    __syncthreads();
    return scratch[warp] + inc - v;
}

// Walks a histogram from its highest bin down and finds the bin that holds the
// `want`-th entry (1-based).  On return (all threads): bin, and `want` reduced by
// the entries in the bins above it.
__device__ void find_bin(const uint32_t* hist, int nbins, uint32_t& want, uint32_t& bin, uint32_t* scratch,
                         uint32_t* result) {
    const int per = nbins / kThreads;  // 8 or 4
    // thread t owns bins [nbins - 1 - t*per - (per - 1), nbins - 1 - t*per], highest first
    uint32_t c[8];
    uint32_t sum = 0;
#pragma unroll
    for (int i = 0; i < 8; ++i)  // all loads in flight together
        c[i] = i < per ? __ldcg(hist + (nbins - 1 - (threadIdx.x * per + i))) : 0u;
#pragma unroll
    for (int i = 0; i < 8; ++i) sum += c[i];
    const uint32_t before = block_exclusive_scan(sum, scratch);
    if (before < want && want <= before + sum) {
        uint32_t run = before;
        bool found = false;
#pragma unroll
        for (int i = 0; i < 8; ++i) {
            if (!found && i < per && want <= run + c[i]) {
                result[0] = nbins - 1 - (threadIdx.x * per + i);
                result[1] = want - run;
                found = true;
            }
            run += c[i];
        }
    }
    __syncthreads();
    bin = result[0];
    want = result[1];
    __syncthreads();
}

// After a histogram pass: the last CTA to get here resolves digit `pass` of the threshold from the finished
// histogram and publishes (prefix, rank left) in the status block.  Every thread of the CTA must call it, after
// its last atomic on the histogram.  `prefix_in`, `want_in`: the state before this digit.
__device__ void publish_digit(StatusBlock* status, const uint32_t* hist, int pass, uint32_t prefix_in, uint32_t want_in,
                              uint32_t* scratch, uint32_t* result) {
    __shared__ uint32_t last_s;
    __threadfence();  // this thread's histogram atomics are ordered before the ticket
    __syncthreads();
    if (threadIdx.x == 0) last_s = atomicAdd(&status->sel_done[pass], 1u) == gridDim.x - 1;
    __syncthreads();
    if (!last_s) return;
    __threadfence();
    uint32_t want = want_in, bin;
    find_bin(hist + pass * kSelBins, pass == 2 ? 1024 : kSelBins, want, bin, scratch, result);
    if (threadIdx.x == 0) {
        status->sel_prefix[pass] = prefix_in | (pass == 0 ? bin << 21 : pass == 1 ? bin << 10 : bin);
        status->sel_want[pass] = want;
    }
}

// Resolves the digits of the threshold key that passes [0, upto) fixed.
// Returns the key prefix (digits placed, lower bits zero) and the rank left
// inside that prefix.
__device__ uint32_t resolve_prefix(const uint32_t* hist, int upto, uint32_t k, uint32_t& want, uint32_t* scratch,
                                   uint32_t* result) {
    uint32_t prefix = 0;
    want = k;
    for (int p = 0; p < upto; ++p) {
        uint32_t bin;
        find_bin(hist + p * kSelBins, p == 2 ? 1024 : kSelBins, want, bin, scratch, result);
        prefix |= p == 0 ? bin << 21 : p == 1 ? bin << 10 : bin;
    }
    return prefix;
}

__device__ __forceinline__ uint32_t prefix_mask(int pass) { return pass == 0 ? 0u : pass == 1 ? 0xFFE00000u : 0xFFFFFC00u; }

// Loads the 16 keys thread `threadIdx.x` owns in tile `tile` (consecutive
// indices), 0 beyond N.  Key 0 belongs to no loss (loss_key never returns it).
__device__ __forceinline__ void load_keys(const float* __restrict__ losses, int64_t N, int64_t base, uint32_t (&key)[kPerThread]) {
    if (base + kPerThread <= N && (reinterpret_cast<uintptr_t>(losses + base) & 15) == 0) {
        float4 q[kPerThread / 4];
#pragma unroll
        for (int i = 0; i < kPerThread / 4; ++i) q[i] = reinterpret_cast<const float4*>(losses + base)[i];
#pragma unroll
        for (int i = 0; i < kPerThread / 4; ++i) {
            key[4 * i] = loss_key(q[i].x);
            key[4 * i + 1] = loss_key(q[i].y);
            key[4 * i + 2] = loss_key(q[i].z);
            key[4 * i + 3] = loss_key(q[i].w);
        }
        return;
    }
#pragma unroll
    for (int i = 0; i < kPerThread; ++i) {
        const int64_t j = base + i;
        key[i] = j < N ? loss_key(losses[j]) : 0u;
    }
}

// Histogram pass `pass`: counts digit `pass` of the keys that match the prefix fixed by the earlier passes, then
// (last CTA) resolves that digit.  `prev_published`: the state after the previous pass is in the status block;
// otherwise (pass 1 after a scorer that built the first histogram itself) digit 0 is resolved here by every CTA.
__global__ void __launch_bounds__(kThreads)
select_hist_kernel(const float* __restrict__ losses, int64_t N, uint32_t k, int pass, bool prev_published,
                   uint32_t* hist, StatusBlock* status) {
    __shared__ uint32_t hist_s[kSelBins];
    __shared__ uint32_t scratch[kThreads / 32 + 1];
    __shared__ uint32_t result[2];
    for (int i = threadIdx.x; i < kSelBins; i += kThreads) hist_s[i] = 0;
    grid_dependency_wait();
    uint32_t want = k, prefix = 0;
    if (pass > 0) {
        if (prev_published) {
            prefix = __ldcg(&status->sel_prefix[pass - 1]);
            want = __ldcg(&status->sel_want[pass - 1]);
        } else {
            prefix = resolve_prefix(hist, pass, k, want, scratch, result);
        }
    }
    __syncthreads();
    const uint32_t mask = prefix_mask(pass);
    for (int64_t tile = blockIdx.x; tile * kTile < N; tile += gridDim.x) {
        const int64_t base = tile * kTile;
        float v[kPerThread];
#pragma unroll
        for (int i = 0; i < kPerThread; ++i) {  // all loads first: they are independent
            const int64_t j = base + i * kThreads + threadIdx.x;
            v[i] = j < N ? losses[j] : 0.f;
        }
#pragma unroll
        for (int i = 0; i < kPerThread; ++i) {
            const int64_t j = base + i * kThreads + threadIdx.x;
            const uint32_t key = loss_key(v[i]);
            const bool in = j < N && (key & mask) == prefix;
            if (pass == 0) {
                // every key counts and losses crowd into a few bins: one atomic per distinct digit and warp
                const uint32_t d = in ? digit_of(key, 0) : 0xFFFFFFFFu;
                const uint32_t peers = __match_any_sync(0xFFFFFFFFu, d);
                if (in && (threadIdx.x & 31) == __ffs(peers) - 1) atomicAdd(&hist_s[d], __popc(peers));
            } else if (in) {
                atomicAdd(&hist_s[digit_of(key, pass)], 1u);
            }
        }
    }
    __syncthreads();
    grid_launch_dependents();  // only the flush and the digit's resolution are left
    uint32_t* out = hist + pass * kSelBins;
    for (int i = threadIdx.x; i < kSelBins; i += kThreads)
        if (hist_s[i]) atomicAdd(&out[i], hist_s[i]);
    publish_digit(status, hist, pass, prefix, want, scratch, result);
}

// Per tile: how many keys are above the threshold, how many equal it.
__global__ void __launch_bounds__(kThreads)
select_count_kernel(const float* __restrict__ losses, int64_t N, const StatusBlock* status, uint32_t* tile_counts) {
    __shared__ uint32_t cnt[2];
    grid_dependency_wait();
    const uint32_t T = __ldcg(&status->sel_prefix[kSelPasses - 1]);
    for (int64_t tile = blockIdx.x; tile * kTile < N; tile += gridDim.x) {
        if (threadIdx.x < 2) cnt[threadIdx.x] = 0;
        __syncthreads();
        uint32_t gt = 0, eq = 0;
        float v[kPerThread];
#pragma unroll
        for (int i = 0; i < kPerThread; ++i) {
            const int64_t j = tile * kTile + i * kThreads + threadIdx.x;
            v[i] = j < N ? losses[j] : 0.f;
        }
#pragma unroll
        for (int i = 0; i < kPerThread; ++i) {
            const int64_t j = tile * kTile + i * kThreads + threadIdx.x;
            const uint32_t key = j < N ? loss_key(v[i]) : 0u;  // key 0 belongs to no loss and is below every threshold
            gt += key > T;
            eq += key == T;
        }
        gt = warp_sum(static_cast<int>(gt));
        eq = warp_sum(static_cast<int>(eq));
        if ((threadIdx.x & 31) == 0) {
            atomicAdd(&cnt[0], gt);
            atomicAdd(&cnt[1], eq);
        }
        __syncthreads();
        if (threadIdx.x < 2) tile_counts[2 * tile + threadIdx.x] = cnt[threadIdx.x];
        __syncthreads();
        if (tile + gridDim.x >= (N + kTile - 1) / kTile) grid_launch_dependents();  // this CTA's last tile is done
    }
}

// Emit: keeps every key above the threshold and the first `r` (by index) equal
// to it, in index order.  Positions come from the tile counts and an in-tile
// scan.  DIRECT: write the final index-ascending result; otherwise write the
// (key, index) pairs for the sort and count their first sort digit.
template <bool DIRECT>
__global__ void __launch_bounds__(kThreads)
select_emit_kernel(const float* __restrict__ losses, int64_t N, const StatusBlock* status,
                   const uint32_t* tile_counts, int32_t* __restrict__ out_idx,
                   float* __restrict__ out_vals, uint32_t* __restrict__ out_keys, uint32_t* __restrict__ tile_hist,
                   int sort_shift) {
    __shared__ uint32_t scratch[kThreads / 32 + 1];
    __shared__ uint32_t pre[2];
    grid_dependency_wait();
    const uint32_t T = __ldcg(&status->sel_prefix[kSelPasses - 1]);
    const uint32_t r = __ldcg(&status->sel_want[kSelPasses - 1]);
    for (int64_t tile = blockIdx.x; tile * kTile < N; tile += gridDim.x) {
        // entries above / equal to the threshold in the tiles before this one
        if (threadIdx.x < 2) pre[threadIdx.x] = 0;
        __syncthreads();
        uint32_t gt = 0, eq = 0;
        for (int64_t t = threadIdx.x; t < tile; t += kThreads) {
            gt += __ldcg(tile_counts + 2 * t);
            eq += __ldcg(tile_counts + 2 * t + 1);
        }
        gt = warp_sum(static_cast<int>(gt));
        eq = warp_sum(static_cast<int>(eq));
        if ((threadIdx.x & 31) == 0) {
            atomicAdd(&pre[0], gt);
            atomicAdd(&pre[1], eq);
        }
        __syncthreads();
        const uint32_t gt_before = pre[0], eq_before = pre[1];

        const int64_t base = tile * kTile + static_cast<int64_t>(threadIdx.x) * kPerThread;
        uint32_t key[kPerThread];
        load_keys(losses, N, base, key);
        if (tile + gridDim.x >= (N + kTile - 1) / kTile) grid_launch_dependents();  // this CTA's last tile
        uint32_t my_gt = 0, my_eq = 0;
#pragma unroll
        for (int i = 0; i < kPerThread; ++i) {
            my_gt += key[i] > T;
            my_eq += (key[i] == T);
        }
        // one scan for both counts: each is at most kTile = 4096 < 2^16
        const uint32_t packed = block_exclusive_scan(my_gt | (my_eq << 16), scratch);
        uint32_t gt_run = gt_before + (packed & 0xFFFFu);
        uint32_t eq_run = eq_before + (packed >> 16);
#pragma unroll
        for (int i = 0; i < kPerThread; ++i) {
            const bool above = key[i] > T;
            const bool tie = key[i] == T;
            if (above || (tie && eq_run < r)) {
                const uint32_t pos = gt_run + min(eq_run, r);
                const int64_t j = base + i;
                if (DIRECT) {
                    out_idx[pos] = static_cast<int32_t>(j);
                    if (out_vals) out_vals[pos] = losses[j];
                } else {
                    out_idx[pos] = static_cast<int32_t>(j);
                    out_keys[pos] = key[i];
                    atomicAdd(&tile_hist[(pos >> sort_shift) * kSortBins + (255u - (key[i] & 0xFFu))], 1u);
                }
            }
            gt_run += above;
            eq_run += tie;
        }
        __syncthreads();
    }
}

// Lanes of the warp whose 8-bit digit equals this lane's, among the lanes with `live` set (0 for a lane that is
// not live).  Nine votes; cheaper here than the generic match instruction.
__device__ __forceinline__ uint32_t match_digit8(uint32_t d, bool live) {
    uint32_t peers = __ballot_sync(0xFFFFFFFFu, live);
#pragma unroll
    for (int b = 0; b < 8; ++b) {
        const bool bit = (d >> b) & 1u;
        const uint32_t m = __ballot_sync(0xFFFFFFFFu, bit);
        peers &= bit ? m : ~m;
    }
    return live ? peers : 0u;
}

// One stable LSD pass over the selected pairs, on digit `pass` (8 bits, least
// significant first), larger digits first.  Reads the digit counts per source
// tile, ranks the tile's entries stably (warp match + per-warp counters), and
// scatters.  Unless LAST, also counts the next digit per destination tile.
// The pass is latency-bound (a short chain of dependent steps per tile), so a
// tile is spread over 32 warps: four ranking rounds per warp instead of sixteen.
constexpr int kSortThreads = 1024;

template <bool LAST, int kRounds>  // kRounds rounds of 32 consecutive entries per warp: tiles of 1024 kRounds entries
__global__ void __launch_bounds__(kSortThreads)
sort_scatter_kernel(const uint32_t* __restrict__ keys_in, const int32_t* __restrict__ idx_in, uint32_t k, int pass,
                    const uint32_t* __restrict__ tile_hist, uint32_t* __restrict__ keys_out,
                    int32_t* __restrict__ idx_out, uint32_t* __restrict__ next_hist,
                    const float* __restrict__ losses, float* __restrict__ out_vals) {
    constexpr int kWarps = kSortThreads / 32;
    constexpr uint32_t kSortTile = kSortThreads * kRounds;
    constexpr int kSortShift = kRounds == 1 ? 10 : 12;
    static_assert(kRounds == 1 || kRounds == 4, "tiles of 1024 or 4096 entries");
    static_assert(kSortBins == 256 && kSortThreads >= kSortBins, "one thread per digit in the scans");
    __shared__ uint32_t counters[kWarps][kSortBins];
    __shared__ uint32_t base_s[kSortBins];
    __shared__ uint32_t tot_s[kSortBins];
    constexpr int kParts = kSortThreads / kSortBins;
    __shared__ uint32_t part_tot[kParts][kSortBins], part_bef[kParts][kSortBins];
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const uint32_t tiles = (k + kSortTile - 1) / kSortTile;
    const int shift = 8 * pass;
    grid_dependency_wait();
    for (uint32_t tile = blockIdx.x; tile < tiles; tile += gridDim.x) {
        // where each digit's run starts for this tile: all entries of earlier digits, plus
        // this digit's entries in earlier tiles
        // (four threads per digit, each over a quarter of the tiles: the chain of dependent loads is what a
        // pass with many tiles waits for)
        {
            const int d = tid & (kSortBins - 1), q = tid / kSortBins;
            const uint32_t per = (tiles + kParts - 1) / kParts;
            const uint32_t t_lo = q * per, t_hi = min(tiles, t_lo + per);
            uint32_t total = 0, bef = 0;
            for (uint32_t t0 = t_lo; t0 < t_hi; t0 += 8) {
                uint32_t c[8];
#pragma unroll
                for (int u = 0; u < 8; ++u)  // eight independent loads in flight
                    c[u] = t0 + u < t_hi ? __ldcg(tile_hist + (t0 + u) * kSortBins + d) : 0u;
#pragma unroll
                for (int u = 0; u < 8; ++u) {
                    total += c[u];
                    bef += t0 + u < tile ? c[u] : 0u;
                }
            }
            part_tot[q][d] = total;
            part_bef[q][d] = bef;
        }
#pragma unroll
        for (int i = 0; i < kWarps * kSortBins / kSortThreads; ++i) (&counters[0][0])[i * kSortThreads + tid] = 0;
        uint32_t key[kRounds], rank[kRounds];
        int32_t idx[kRounds];
        const uint32_t first = tile * kSortTile + warp * (kRounds * 32);
#pragma unroll
        for (int rd = 0; rd < kRounds; ++rd) {  // all loads first: they are independent
            const uint32_t e = first + rd * 32 + lane;
            key[rd] = e < k ? __ldcg(keys_in + e) : 0u;
            idx[rd] = e < k ? __ldcg(idx_in + e) : 0;
        }
        __syncthreads();
        uint32_t before = 0;
        if (tid < kSortBins) {
            uint32_t total = 0;
#pragma unroll
            for (int q = 0; q < kParts; ++q) {
                total += part_tot[q][tid];
                before += part_bef[q][tid];
            }
            tot_s[tid] = total;
        }
        __syncthreads();
        if (warp == 0) {  // exclusive scan of the 256 digit totals, eight per lane
            uint32_t v[8], sum = 0;
#pragma unroll
            for (int i = 0; i < 8; ++i) {
                v[i] = tot_s[lane * 8 + i];
                sum += v[i];
            }
            uint32_t inc = sum;
#pragma unroll
            for (int o = 1; o < 32; o <<= 1) {
                const uint32_t n = __shfl_up_sync(0xFFFFFFFFu, inc, o);
                if (lane >= o) inc += n;
            }
            uint32_t run = inc - sum;
#pragma unroll
            for (int i = 0; i < 8; ++i) {
                tot_s[lane * 8 + i] = run;
                run += v[i];
            }
        }
#pragma unroll
        for (int rd = 0; rd < kRounds; ++rd) {
            const uint32_t e = first + rd * 32 + lane;
            const bool live = e < k;
            const uint32_t dd = 255u - ((key[rd] >> shift) & 0xFFu);
            const uint32_t peers = match_digit8(dd, live);
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
        __syncthreads();
        if (tid < kSortBins) {
            base_s[tid] = tot_s[tid] + before;
            uint32_t run = 0;
#pragma unroll
            for (int w = 0; w < kWarps; ++w) {
                const uint32_t c = counters[w][tid];
                counters[w][tid] = run;
                run += c;
            }
        }
        __syncthreads();
        if (tile + gridDim.x >= tiles) grid_launch_dependents();  // only this CTA's last scatter is left
#pragma unroll
        for (int rd = 0; rd < kRounds; ++rd) {
            const uint32_t e = first + rd * 32 + lane;
            const bool live = e < k;
            uint32_t pos = 0;
            if (live) {
                const uint32_t dd = 255u - ((key[rd] >> shift) & 0xFFu);
                pos = base_s[dd] + counters[warp][dd] + rank[rd];
                idx_out[pos] = idx[rd];
                if (LAST) {
                    if (out_vals) out_vals[pos] = losses[idx[rd]];
                } else {
                    keys_out[pos] = key[rd];
                }
            }
            if (!LAST) {
                // count the next digit per destination tile.  High digits are nearly constant over the selection,
                // so a warp sends one atomic per distinct counter instead of one per entry.
                const uint32_t nd = 255u - ((key[rd] >> (shift + 8)) & 0xFFu);
                const uint32_t peers = match_digit8(nd, live);
                const int leader = live ? __ffs(peers) - 1 : lane;
                const uint32_t t = pos >> kSortShift;
                const bool with_leader = t == __shfl_sync(0xFFFFFFFFu, t, leader);  // same destination tile as the leader
                const uint32_t same = __ballot_sync(0xFFFFFFFFu, live && with_leader);
                if (live) {
                    if (lane == leader) atomicAdd(&next_hist[t * kSortBins + nd], static_cast<uint32_t>(__popc(peers & same)));
                    else if (!with_leader) atomicAdd(&next_hist[t * kSortBins + nd], 1u);
                }
            }
        }
        __syncthreads();
    }
}

// Small pools: one CTA sorts all N composite keys (key, ~index), one per thread, with a
// bitonic network; the first k are the selection in loss-descending order.
constexpr int kSmallThreads = 1024;

__global__ void __launch_bounds__(kSmallThreads)
small_topk_kernel(const float* __restrict__ losses, int n, int k, int order, int32_t* __restrict__ out_idx,
                  float* __restrict__ out_vals) {
    __shared__ unsigned long long ck[kSmallN];
    __shared__ uint32_t warp_tot[kSmallThreads / 32];
    grid_dependency_wait();
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
    constexpr int kPer = 1;  // one index per thread
    const int base = threadIdx.x * kPer;
    bool sel[kPer];
    uint32_t mine = 0;
#pragma unroll
    for (int i = 0; i < kPer; ++i) {
        const int j = base + i;
        sel[i] = j < n && ((static_cast<unsigned long long>(loss_key(losses[j])) << 32) | (0xFFFFFFFFu - static_cast<uint32_t>(j))) >= cut;
        mine += sel[i];
    }
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    uint32_t inc = mine;
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) {
        const uint32_t v = __shfl_up_sync(0xFFFFFFFFu, inc, o);
        if (lane >= o) inc += v;
    }
    if (lane == 31) warp_tot[warp] = inc;
    __syncthreads();
    uint32_t pos = inc - mine;
    for (int w = 0; w < warp; ++w) pos += warp_tot[w];
#pragma unroll
    for (int i = 0; i < kPer; ++i)
        if (sel[i]) {
            out_idx[pos] = base + i;
            if (out_vals) out_vals[pos] = losses[base + i];
            ++pos;
        }
}

}  // namespace

cudaError_t launch_topk(const float* losses, int64_t N, int64_t k, lsgd_order order, int32_t* out_idx,
                        float* out_vals, const TopkWorkspace& ws, bool hist0_ready, cudaStream_t s) {
    if (N <= kSmallN)
        return launch_dependent(small_topk_kernel, 1, kSmallThreads, s, losses, static_cast<int>(N), static_cast<int>(k),
                                static_cast<int>(order), out_idx, out_vals);
    const int64_t tiles_n = (N + kTile - 1) / kTile;
    const int grid_n = static_cast<int>(std::min<int64_t>(tiles_n, static_cast<int64_t>(sm_count()) * 8));
    const uint32_t kk = static_cast<uint32_t>(k);
    cudaError_t e = cudaSuccess;
    for (int pass = hist0_ready ? 1 : 0; pass < kSelPasses && e == cudaSuccess; ++pass)
        e = launch_dependent(select_hist_kernel, grid_n, kThreads, s, losses, N, kk, pass,
                             pass > (hist0_ready ? 1 : 0), ws.hist, ws.status);
    if (e != cudaSuccess) return e;
    e = launch_dependent(select_count_kernel, grid_n, kThreads, s, losses, N, ws.status, ws.tile_counts);
    if (e != cudaSuccess) return e;
    if (order == LSGD_ORDER_INDEX_ASC)
        return launch_dependent(select_emit_kernel<true>, grid_n, kThreads, s, losses, N, ws.status, ws.tile_counts,
                                out_idx, out_vals, nullptr, nullptr, 12);
    const int sort_shift = sort_tile_shift(k);
    const int64_t tiles_k = static_cast<int64_t>(sort_tiles(k));
    const size_t th = sort_tiles_bound(k) * kSortBins;  // digit counts of one pass
    e = launch_dependent(select_emit_kernel<false>, grid_n, kThreads, s, losses, N, ws.status, ws.tile_counts, ws.idx[0],
                         nullptr, ws.keys[0], ws.tile_hist, sort_shift);
    const int grid_k = static_cast<int>(std::min<int64_t>(tiles_k, static_cast<int64_t>(sm_count()) * 2));
    auto pass_kernel = [&](auto mid, auto last) {
        for (int pass = 0; pass < 3 && e == cudaSuccess; ++pass)
            e = launch_dependent(mid, grid_k, kSortThreads, s, ws.keys[pass & 1], ws.idx[pass & 1], kk, pass,
                                 ws.tile_hist + pass * th, ws.keys[(pass + 1) & 1], ws.idx[(pass + 1) & 1],
                                 ws.tile_hist + (pass + 1) * th, nullptr, nullptr);
        if (e != cudaSuccess) return;
        e = launch_dependent(last, grid_k, kSortThreads, s, ws.keys[1], ws.idx[1], kk, 3, ws.tile_hist + 3 * th, nullptr,
                             out_idx, nullptr, losses, out_vals);
    };
    if (sort_shift == 10) pass_kernel(sort_scatter_kernel<false, 1>, sort_scatter_kernel<true, 1>);
    else pass_kernel(sort_scatter_kernel<false, 4>, sort_scatter_kernel<true, 4>);
    return e;
}

}  // namespace lsgd
