// The C ABI of liblsgd (include/lsgd.h): argument checks on the host, then
// stream-ordered launches.  No device memory is allocated here.
#include <atomic>
#include <cstdlib>
#include <cstring>

#include "lsgd_internal.cuh"

namespace lsgd {

int sm_count() {
    static std::atomic<int> cache[64];
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess) return 1;
    std::atomic<int>& c = cache[dev & 63];
    int v = c.load(std::memory_order_relaxed);
    if (v == 0) {
        if (cudaDeviceGetAttribute(&v, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess || v < 1) v = 1;
        c.store(v, std::memory_order_relaxed);
    }
    return v;
}

TestGeometry test_geometry() {
    TestGeometry g{2147483647, false, false, false};
    if (const char* v = std::getenv("LSGD_TEST_MAX_CTAS")) {
        const long n = std::strtol(v, nullptr, 10);
        if (n > 0 && n < 2147483647) g.max_ctas = static_cast<int>(n);
    }
    if (const char* v = std::getenv("LSGD_TEST_NO_CLUSTER")) g.no_cluster = v[0] == '1';
    if (const char* v = std::getenv("LSGD_TEST_NARROW_CLUSTER")) g.narrow_cluster = v[0] == '1';
    if (const char* v = std::getenv("LSGD_TEST_PHANTOM_BLOCK")) g.phantom_block = v[0] == '1';
    return g;
}

size_t score_workspace_bytes(int64_t N, int64_t T, int64_t C) {
    if (N < 0 || T < 1 || C < 1) return 0;
    return sizeof(StatusBlock) + (T > 1 ? align_up(sizeof(float) * static_cast<size_t>(N) * static_cast<size_t>(T)) : 0);
}

ScoreWorkspace carve_score(void* ws, int64_t, int64_t, int64_t) {
    ScoreWorkspace w;
    w.status = static_cast<StatusBlock*>(ws);
    w.token_loss = reinterpret_cast<float*>(static_cast<unsigned char*>(ws) + sizeof(StatusBlock));
    return w;
}

namespace {

bool aligned(const void* p, size_t a) { return (reinterpret_cast<uintptr_t>(p) & (a - 1)) == 0; }

bool overlaps(const void* a, size_t na, const void* b, size_t nb) {
    const uintptr_t a0 = reinterpret_cast<uintptr_t>(a), b0 = reinterpret_cast<uintptr_t>(b);
    return a0 < b0 + nb && b0 < a0 + na;
}

lsgd_status check_pool(const void* logits, int dtype, const int64_t* labels, int64_t N, int64_t T, int64_t C,
                       const float* losses) {
    if (dtype != LSGD_F32 && dtype != LSGD_BF16) return LSGD_ERR_UNSUPPORTED;
    if (N < 0 || T < 1 || C < 1) return LSGD_ERR_INVALID_ARG;
    if (N >= (int64_t{1} << 31) || C >= (int64_t{1} << 31)) return LSGD_ERR_UNSUPPORTED;
    if (N > 0 && T > (int64_t{1} << 62) / N) return LSGD_ERR_UNSUPPORTED;
    if (N == 0) return LSGD_OK;
    if (!logits || !labels || !losses) return LSGD_ERR_INVALID_ARG;
    const size_t es = dtype == LSGD_F32 ? 4 : 2;
    if (!aligned(logits, es) || !aligned(labels, 8) || !aligned(losses, 4)) return LSGD_ERR_ALIGNMENT;
    if (overlaps(logits, es * static_cast<size_t>(N) * T * C, losses, sizeof(float) * static_cast<size_t>(N)))
        return LSGD_ERR_INVALID_ARG;
    return LSGD_OK;
}

lsgd_status check_topk(const float* losses, int64_t N, int64_t k, int order, const int32_t* out_idx,
                       const float* out_vals) {
    if (order != LSGD_ORDER_LOSS_DESC && order != LSGD_ORDER_INDEX_ASC) return LSGD_ERR_UNSUPPORTED;
    if (N < 0 || k < 0 || k > N) return LSGD_ERR_INVALID_ARG;
    if (N >= (int64_t{1} << 31)) return LSGD_ERR_UNSUPPORTED;
    if (k == 0) return LSGD_OK;
    if (!losses || !out_idx) return LSGD_ERR_INVALID_ARG;
    if (!aligned(losses, 4) || !aligned(out_idx, 4) || (out_vals && !aligned(out_vals, 4))) return LSGD_ERR_ALIGNMENT;
    return LSGD_OK;
}

lsgd_status check_ws(const void* ws, size_t have, size_t need) {
    if (!ws) return LSGD_ERR_INVALID_ARG;
    if (!aligned(ws, kAlign)) return LSGD_ERR_ALIGNMENT;
    if (have < need) return LSGD_ERR_WORKSPACE;
    return LSGD_OK;
}

inline lsgd_status from_cuda(cudaError_t e) { return e == cudaSuccess ? LSGD_OK : LSGD_ERR_CUDA; }

}  // namespace
}  // namespace lsgd

using namespace lsgd;

extern "C" {

int lsgd_version(void) { return 100; }

const char* lsgd_status_string(int status) {
    switch (status) {
        case LSGD_OK: return "ok";
        case LSGD_ERR_INVALID_ARG: return "invalid argument";
        case LSGD_ERR_UNSUPPORTED: return "unsupported dtype, order or size";
        case LSGD_ERR_ALIGNMENT: return "misaligned pointer";
        case LSGD_ERR_WORKSPACE: return "workspace too small";
        case LSGD_ERR_CUDA: return "CUDA runtime error";
        case LSGD_ERR_TIMEOUT: return "device-side wait timed out";
        default: return "unknown status";
    }
}

size_t lsgd_score_workspace_bytes(int64_t N, int64_t T, int64_t C) { return score_workspace_bytes(N, T, C); }

size_t lsgd_topk_workspace_bytes(int64_t N, int64_t k) { return topk_workspace_bytes(N, k); }

size_t lsgd_score_topk_workspace_bytes(int64_t N, int64_t T, int64_t C, int64_t k) {
    const size_t a = topk_workspace_bytes(N, k), b = score_workspace_bytes(N, T, C);
    return (a && b) ? a + (b - sizeof(StatusBlock)) : 0;
}

lsgd_status lsgd_score_losses(const void* logits, lsgd_dtype dtype, const int64_t* labels, int64_t N, int64_t T,
                              int64_t C, int64_t ignore_index, float* losses, void* ws, size_t ws_bytes,
                              void* cuda_stream) {
    lsgd_status st = check_pool(logits, dtype, labels, N, T, C, losses);
    if (st != LSGD_OK || N == 0) return st;
    st = check_ws(ws, ws_bytes, score_workspace_bytes(N, T, C));
    if (st != LSGD_OK) return st;
    cudaStream_t s = static_cast<cudaStream_t>(cuda_stream);
    cudaError_t e = clear_device_words(ws, sizeof(StatusBlock), s);
    if (e != cudaSuccess) return LSGD_ERR_CUDA;
    return from_cuda(launch_score(logits, dtype, labels, N, T, C, ignore_index, losses, carve_score(ws, N, T, C),
                                  nullptr, s));
}

lsgd_status lsgd_topk_select(const float* losses, int64_t N, int64_t k, lsgd_order order, int32_t* out_idx,
                             float* out_vals, void* ws, size_t ws_bytes, void* cuda_stream) {
    lsgd_status st = check_topk(losses, N, k, order, out_idx, out_vals);
    if (st != LSGD_OK || k == 0) return st;
    st = check_ws(ws, ws_bytes, topk_workspace_bytes(N, k));
    if (st != LSGD_OK) return st;
    cudaStream_t s = static_cast<cudaStream_t>(cuda_stream);
    return from_cuda(launch_topk(losses, N, k, order, out_idx, out_vals, carve_topk(ws, N, k), false, true, s));
}

lsgd_status lsgd_score_topk(const void* logits, lsgd_dtype dtype, const int64_t* labels, int64_t N, int64_t T,
                            int64_t C, int64_t ignore_index, int64_t k, lsgd_order order, float* losses,
                            int32_t* out_idx, float* out_vals, void* ws, size_t ws_bytes, void* cuda_stream) {
    lsgd_status st = check_pool(logits, dtype, labels, N, T, C, losses);
    if (st != LSGD_OK) return st;
    st = check_topk(losses, N, k, order, out_idx, out_vals);
    if (st != LSGD_OK || N == 0) return st;
    if (k > 0 && (overlaps(out_idx, 4 * static_cast<size_t>(k), losses, 4 * static_cast<size_t>(N)) ||
                  (out_vals && overlaps(out_vals, 4 * static_cast<size_t>(k), losses, 4 * static_cast<size_t>(N)))))
        return LSGD_ERR_INVALID_ARG;
    st = check_ws(ws, ws_bytes, lsgd_score_topk_workspace_bytes(N, T, C, k));
    if (st != LSGD_OK) return st;
    cudaStream_t s = static_cast<cudaStream_t>(cuda_stream);
    if (zero_topk_workspace(ws, k, s) != cudaSuccess) return LSGD_ERR_CUDA;
    const TopkWorkspace tw = carve_topk(ws, N, k);
    ScoreWorkspace sw;
    sw.status = tw.status;
    sw.token_loss = reinterpret_cast<float*>(static_cast<unsigned char*>(ws) + topk_workspace_bytes(N, k));
    // the scorer (or the sequence mean) feeds the first radix histogram unless one CTA sorts the whole pool
    const bool fuse_hist = k > 0 && N > kSmallN;
    cudaError_t e = launch_score(logits, dtype, labels, N, T, C, ignore_index, losses, sw,
                                 fuse_hist ? tw.hist : nullptr, s);
    if (e != cudaSuccess) return LSGD_ERR_CUDA;
    if (k == 0) return LSGD_OK;
    return from_cuda(launch_topk(losses, N, k, order, out_idx, out_vals, tw, fuse_hist, false, s));
}

lsgd_status lsgd_aggregate(const float* const* replicas, const float* weights, int32_t P, int64_t D, float* out,
                           void* cuda_stream) {
    if (P < 1 || P > LSGD_MAX_REPLICAS || D < 0) return LSGD_ERR_INVALID_ARG;
    if (!replicas || !weights) return LSGD_ERR_INVALID_ARG;
    if (D == 0) return LSGD_OK;
    if (!out) return LSGD_ERR_INVALID_ARG;
    bool vec = aligned(out, 16);
    const size_t bytes = sizeof(float) * static_cast<size_t>(D);
    for (int i = 0; i < P; ++i) {
        if (!replicas[i]) return LSGD_ERR_INVALID_ARG;
        if (!aligned(replicas[i], 4)) return LSGD_ERR_ALIGNMENT;
        vec = vec && aligned(replicas[i], 16);
        if (replicas[i] != out && overlaps(replicas[i], bytes, out, bytes)) return LSGD_ERR_INVALID_ARG;
    }
    if (!aligned(out, 4)) return LSGD_ERR_ALIGNMENT;
    return from_cuda(launch_aggregate(replicas, weights, P, D, out, vec, static_cast<cudaStream_t>(cuda_stream)));
}

lsgd_status lsgd_weights_from_steps(const int32_t* tau, int32_t P, float* w_out) {
    if (!tau || !w_out || P < 1) return LSGD_ERR_INVALID_ARG;
    int64_t total = 0;
    for (int i = 0; i < P; ++i) {
        if (tau[i] < 0) return LSGD_ERR_INVALID_ARG;
        total += tau[i];
    }
    if (total <= 0) return LSGD_ERR_INVALID_ARG;
    for (int i = 0; i < P; ++i) w_out[i] = static_cast<float>(static_cast<double>(tau[i]) / static_cast<double>(total));
    return LSGD_OK;
}

lsgd_status lsgd_read_device_status(const void* ws, int32_t* bad_label_count, void* cuda_stream) {
    if (!ws || !bad_label_count) return LSGD_ERR_INVALID_ARG;
    StatusBlock sb;
    cudaStream_t s = static_cast<cudaStream_t>(cuda_stream);
    if (cudaMemcpyAsync(&sb, ws, sizeof sb, cudaMemcpyDeviceToHost, s) != cudaSuccess) return LSGD_ERR_CUDA;
    if (cudaStreamSynchronize(s) != cudaSuccess) return LSGD_ERR_CUDA;
    *bad_label_count = sb.bad_labels;
    return sb.timeout ? LSGD_ERR_TIMEOUT : LSGD_OK;
}

}  // extern "C"
