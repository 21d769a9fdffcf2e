// extern "C" boundary: argument checks, workspace carving, dispatch.  See include/vocabtrim.h
// for the contract of every entry point.
#include <atomic>

#include "vt_common.cuh"

#include <cmath>
#include <cstdint>

namespace vt {

static std::atomic<uint64_t> g_launches{0};
void count_launch(int n) { g_launches.fetch_add((uint64_t)n, std::memory_order_relaxed); }

int num_sms() {
    static int cached[64] = {0};
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess) return kNumSMsFallback;
    if (dev >= 0 && dev < 64 && cached[dev]) return cached[dev];
    int n = 0;
    if (cudaDeviceGetAttribute(&n, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess || n <= 0)
        n = kNumSMsFallback;
    if (dev >= 0 && dev < 64) cached[dev] = n;
    return n;
}

namespace {

inline bool aligned(const void* p, size_t a) { return (reinterpret_cast<uintptr_t>(p) % a) == 0; }
inline cudaStream_t as_stream(void* s) { return reinterpret_cast<cudaStream_t>(s); }
thread_local cudaError_t t_last_cuda = cudaSuccess;
inline vt_status from_cuda(cudaError_t e) {
    if (e == cudaSuccess) return VT_OK;
    t_last_cuda = e;
    return VT_ERR_CUDA;
}

constexpr int64_t kHostChunkIds = 1 << 24;     // ids per staged chunk of vt_build_vocab_host

bool hist_shape_ok(int32_t V) { return hist_supported(V); }

bool head_shape_ok(int32_t B, int32_t K, int32_t d, int32_t topk) {
    if (B < 1 || B > 256 || K < 1 || d < 8 || (d & 7) || topk < 1 || topk > VT_MAX_TOPK || topk > K)
        return false;
    return head_skinny_supported(B, d) || (head_dense_supported(B, K, d) && head_dense_topk_ok(topk));
}

size_t head_scratch(int32_t B, int32_t K, int32_t d, int32_t topk) {
    if (head_skinny_supported(B, d)) return head_skinny_scratch_bytes(B, K, topk);
    return head_dense_scratch_bytes(B, K, topk);
}

// staging layout of vt_draft_head_host after the head scratch
struct HostStage {
    size_t off_h, off_temp, off_u, off_ids, off_lp, bytes;
};
HostStage host_stage(int32_t B, int32_t K, int32_t d, int32_t topk, size_t base) {
    HostStage s{};
    size_t o = align_up(base, 256);
    s.off_h = o;     o += align_up((size_t)B * d * 2, 256);
    s.off_temp = o;  o += align_up((size_t)B * 4, 256);
    s.off_u = o;     o += align_up((size_t)B * K * 4, 256);
    s.off_ids = o;   o += align_up((size_t)B * (1 + topk) * 4, 256);
    s.off_lp = o;    o += align_up((size_t)B * (1 + topk) * 4, 256);
    s.bytes = o;
    return s;
}

vt_status check_ws(void* ws, size_t ws_bytes, size_t need) {
    if (!ws || !aligned(ws, 256) || need == 0 || ws_bytes < need) return VT_ERR_WORKSPACE;
    return VT_OK;
}

}  // namespace
}  // namespace vt

using namespace vt;

extern "C" {

size_t vt_workspace_bytes(int op, int64_t n, int32_t V, int32_t K, int32_t d, int32_t B,
                          int32_t topk) {
    switch (op) {
        case VT_OP_HISTOGRAM:
            if (!hist_shape_ok(V) || n < 0) return 0;
            return VT_CTRL_BYTES + hist_plan(V).bytes;
        case VT_OP_SELECT_TOPK:
            if (V < 1 || K < 1 || K > V) return 0;
            return VT_CTRL_BYTES + select_cut_scratch_bytes(V);
        case VT_OP_BUILD_VOCAB:
        case VT_OP_BUILD_VOCAB_HOST: {
            if (!hist_shape_ok(V) || n < 0 || K < 1 || K > V) return 0;
            size_t inner = hist_plan(V).bytes;
            if (select_cut_scratch_bytes(V) > inner) inner = select_cut_scratch_bytes(V);
            size_t total = VT_CTRL_BYTES + align_up((size_t)V * 4, 256) + inner;
            if (op == VT_OP_BUILD_VOCAB_HOST) {
                const int64_t chunk = n < kHostChunkIds ? (n > 0 ? n : 1) : kHostChunkIds;
                total = align_up(total, 256) + 2 * align_up((size_t)chunk * 4, 256);
            }
            return total;
        }
        case VT_OP_TRIM_HEAD:
            return VT_CTRL_BYTES;
        case VT_OP_DRAFT_HEAD:
            if (!head_shape_ok(B, K, d, topk)) return 0;
            return VT_CTRL_BYTES + head_scratch(B, K, d, topk);
        case VT_OP_DRAFT_HEAD_HOST:
            if (!head_shape_ok(B, K, d, topk)) return 0;
            return host_stage(B, K, d, topk, VT_CTRL_BYTES + head_scratch(B, K, d, topk)).bytes;
        default:
            return 0;
    }
}

vt_status vt_workspace_init(void* ws, size_t ws_bytes, void* stream) {
    if (!ws || !aligned(ws, 256) || ws_bytes < VT_CTRL_BYTES) return VT_ERR_WORKSPACE;
    return from_cuda(cudaMemsetAsync(ws, 0, VT_CTRL_BYTES, as_stream(stream)));
}

vt_status vt_workspace_set_wait_limit(void* ws, uint64_t nanoseconds, void* stream) {
    if (!ws || !aligned(ws, 256)) return VT_ERR_WORKSPACE;
    Ctrl* dev = static_cast<Ctrl*>(ws);
    const unsigned long long v = nanoseconds;
    cudaStream_t s = as_stream(stream);
    if (cudaMemcpyAsync(&dev->wait_ns, &v, sizeof(v), cudaMemcpyHostToDevice, s) != cudaSuccess) return VT_ERR_CUDA;
    return from_cuda(cudaStreamSynchronize(s));            // `v` lives on this stack frame
}

vt_status vt_read_status(void* ws, void* stream, uint32_t* flags, uint64_t* n_bad) {
    if (!ws) return VT_ERR_WORKSPACE;
    Ctrl host{};
    cudaStream_t s = as_stream(stream);
    if (cudaMemcpyAsync(&host, ws, sizeof(Ctrl), cudaMemcpyDeviceToHost, s) != cudaSuccess)
        return VT_ERR_CUDA;
    if (cudaStreamSynchronize(s) != cudaSuccess) return VT_ERR_CUDA;
    if (host.flags || host.n_bad) {
        // clear the sticky part only (flags + n_bad); tickets are left alone
        Ctrl* dev = static_cast<Ctrl*>(ws);
        if (cudaMemsetAsync(&dev->flags, 0, sizeof(uint32_t), s) != cudaSuccess) return VT_ERR_CUDA;
        if (cudaMemsetAsync(&dev->n_bad, 0, sizeof(unsigned long long), s) != cudaSuccess)
            return VT_ERR_CUDA;
        if (cudaStreamSynchronize(s) != cudaSuccess) return VT_ERR_CUDA;
    }
    if (flags) *flags = host.flags;
    if (n_bad) *n_bad = host.n_bad;
    if (host.flags & VT_FLAG_TIMEOUT) return VT_ERR_TIMEOUT;
    if (host.flags & (VT_FLAG_BAD_ID | VT_FLAG_BAD_MAP)) return VT_ERR_RANGE;
    if (host.flags & (VT_FLAG_BAD_TEMP | VT_FLAG_NAN_ROW)) return VT_ERR_NUMERIC;
    return VT_OK;
}

const char* vt_status_str(vt_status s) {
    switch (s) {
        case VT_OK: return "ok";
        case VT_ERR_INVALID_ARG: return "invalid argument";
        case VT_ERR_RANGE: return "token id or map entry out of range";
        case VT_ERR_WORKSPACE: return "workspace missing, misaligned or too small";
        case VT_ERR_CUDA: return "CUDA runtime error";
        case VT_ERR_TIMEOUT: return "bounded device-side wait expired";
        case VT_ERR_UNSUPPORTED: return "unsupported shape";
        case VT_ERR_NUMERIC: return "non-positive temperature or NaN row";
        default: return "unknown status";
    }
}

#ifdef VT_STAMPS
int32_t vt_stamps_region(int32_t B, int32_t d, int32_t topk, size_t* offset, int32_t* slots, int32_t* max_ctas) {
    if (!offset || !slots || !max_ctas) return 0;
    if (head_skinny_supported(B, d)) *offset = VT_CTRL_BYTES + head_skinny_stamps_offset(B, topk);
    else if (head_dense_supported(B, 1, d)) *offset = VT_CTRL_BYTES + head_dense_stamps_offset(B, topk);
    else return 0;
    *slots = 16;
    *max_ctas = 160;
    return 1;
}
#endif

uint64_t vt_launch_count(void) { return g_launches.load(std::memory_order_relaxed); }

const char* vt_last_cuda_error(void) { return cudaGetErrorString(t_last_cuda); }

vt_status vt_histogram(const int32_t* ids, int64_t n, int32_t V, uint32_t* counts, int accumulate,
                       void* ws, size_t ws_bytes, void* stream) {
    if (n < 0 || n >= ((int64_t)1 << 32) || V < 1 || !counts || (n > 0 && !ids)) return VT_ERR_INVALID_ARG;
    if (!aligned(ids, 4) || !aligned(counts, 4)) return VT_ERR_INVALID_ARG;
    if (!hist_shape_ok(V)) return VT_ERR_UNSUPPORTED;
    vt_status st = check_ws(ws, ws_bytes, vt_workspace_bytes(VT_OP_HISTOGRAM, n, V, 0, 0, 0, 0));
    if (st != VT_OK) return st;
    uint8_t* base = static_cast<uint8_t*>(ws);
    return from_cuda(launch_histogram(ids, n, V, counts, accumulate, reinterpret_cast<Ctrl*>(base),
                                      base + VT_CTRL_BYTES, as_stream(stream)));
}

vt_status vt_histogram_folded(const int32_t* ids, int64_t n, int32_t V, int32_t bins, uint32_t* counts, void* stream) {
    if (n < 0 || n >= ((int64_t)1 << 32) || V < 1 || bins < 1 || !counts || (n > 0 && !ids)) return VT_ERR_INVALID_ARG;
    if (!aligned(ids, 4) || !aligned(counts, 4)) return VT_ERR_INVALID_ARG;
    if (bins > VT_FOLDED_MAX_BINS) return VT_ERR_UNSUPPORTED;
    return from_cuda(launch_hist_fold(ids, n, V, bins, counts, as_stream(stream)));
}

vt_status vt_select_topk(const uint32_t* counts, int32_t V, int32_t K, int32_t* map,
                         int32_t* inv_map, void* ws, size_t ws_bytes, void* stream) {
    if (!counts || !map || !inv_map || V < 1 || K < 1 || K > V) return VT_ERR_INVALID_ARG;
    vt_status st = check_ws(ws, ws_bytes, vt_workspace_bytes(VT_OP_SELECT_TOPK, 0, V, K, 0, 0, 0));
    if (st != VT_OK) return st;
    uint8_t* base = static_cast<uint8_t*>(ws);
    return from_cuda(launch_select_topk(counts, V, K, map, inv_map, base + VT_CTRL_BYTES,
                                        as_stream(stream)));
}

static vt_status select_cut_impl(const uint32_t* counts, int32_t V, int mode, double p, uint32_t min_count,
                                 int32_t* map, int32_t* inv_map, int32_t* k_out, void* ws, size_t ws_bytes,
                                 void* stream) {
    if (!counts || !map || !inv_map || !k_out || V < 1) return VT_ERR_INVALID_ARG;
    if (mode == 0 && (!(p > 0.0) || p > 1.0)) return VT_ERR_INVALID_ARG;
    vt_status st = check_ws(ws, ws_bytes, vt_workspace_bytes(VT_OP_SELECT_TOPK, 0, V, V, 0, 0, 0));
    if (st != VT_OK) return st;
    uint8_t* base = static_cast<uint8_t*>(ws);
    return from_cuda(launch_select_cut(counts, V, mode, p, min_count, map, inv_map, k_out, base + VT_CTRL_BYTES,
                                       as_stream(stream)));
}

vt_status vt_select_topp(const uint32_t* counts, int32_t V, double p, int32_t* map, int32_t* inv_map,
                         int32_t* k_out, void* ws, size_t ws_bytes, void* stream) {
    return select_cut_impl(counts, V, 0, p, 0u, map, inv_map, k_out, ws, ws_bytes, stream);
}

vt_status vt_select_minfreq(const uint32_t* counts, int32_t V, uint32_t min_count, int32_t* map,
                            int32_t* inv_map, int32_t* k_out, void* ws, size_t ws_bytes, void* stream) {
    return select_cut_impl(counts, V, 1, 1.0, min_count, map, inv_map, k_out, ws, ws_bytes, stream);
}

static vt_status check_tree_args(int32_t B, int32_t topk, const int32_t* frontier_nodes, const int32_t* pool_token,
                                 const int32_t* pool_parent, const float* pool_score, int32_t pool_base,
                                 int32_t pool_capacity, int32_t n_front, const int32_t* next_frontier) {
    if (!pool_token || !pool_parent || !pool_score || !next_frontier) return VT_ERR_INVALID_ARG;
    if (B < 1 || topk < 1 || pool_base < 0 || n_front < 1) return VT_ERR_INVALID_ARG;
    if (!frontier_nodes && B != 1) return VT_ERR_INVALID_ARG;
    const int64_t n_new = (int64_t)B * topk;
    if (n_new > tree_max_nodes()) return VT_ERR_UNSUPPORTED;
    if (n_front > n_new || pool_base + n_new > pool_capacity) return VT_ERR_INVALID_ARG;
    return VT_OK;
}

vt_status vt_tree_expand(const int32_t* cand_ids, const float* cand_logprobs, int32_t B, int32_t topk,
                         int32_t ld, int32_t col0, const int32_t* frontier_nodes, int32_t* pool_token,
                         int32_t* pool_parent, float* pool_score, int32_t pool_base, int32_t pool_capacity,
                         int32_t n_front, int32_t* next_frontier, void* stream) {
    if (!cand_ids || !cand_logprobs || col0 < 0 || topk < 1 || ld < col0 + topk) return VT_ERR_INVALID_ARG;
    const vt_status st = check_tree_args(B, topk, frontier_nodes, pool_token, pool_parent, pool_score, pool_base,
                                         pool_capacity, n_front, next_frontier);
    if (st != VT_OK) return st;
    const TreeArgs t{frontier_nodes, pool_token, pool_parent, pool_score, pool_base, n_front, next_frontier};
    return from_cuda(launch_tree_expand(cand_ids, cand_logprobs, B, topk, ld, col0, t, as_stream(stream)));
}

vt_status vt_tree_rerank(const int32_t* pool_token, const int32_t* pool_parent, const float* pool_score,
                         int32_t n, int32_t budget, int32_t* out_nodes, int32_t* out_token, int32_t* out_parent,
                         void* stream) {
    if (!pool_token || !pool_parent || !pool_score || !out_nodes || !out_token || !out_parent)
        return VT_ERR_INVALID_ARG;
    if (n < 1 || budget < 1) return VT_ERR_INVALID_ARG;
    if (n > tree_max_nodes()) return VT_ERR_UNSUPPORTED;
    return from_cuda(launch_tree_rerank(pool_token, pool_parent, pool_score, n, budget, out_nodes, out_token,
                                        out_parent, as_stream(stream)));
}

vt_status vt_verify_greedy(const int32_t* token, const int32_t* parent, const int32_t* target, int32_t S,
                           int32_t N, int32_t* n_accept, int32_t* path, int32_t* emitted,
                           uint64_t* tokens_total, void* stream) {
    if (S < 0 || N < 1 || N == INT32_MAX) return VT_ERR_INVALID_ARG;
    if (S > 0 && (!token || !target || !n_accept)) return VT_ERR_INVALID_ARG;
    return from_cuda(launch_verify_greedy(token, parent, target, S, N, n_accept, path, emitted,
                                          reinterpret_cast<unsigned long long*>(tokens_total),
                                          as_stream(stream)));
}

double vt_mbsu(double tau, double draft_params, double target_params, int32_t gamma) {
    if (!(tau >= 0.0) || !(draft_params >= 0.0) || !(target_params > 0.0) || gamma < 0) return nan("");
    const double c = draft_params / target_params;
    return tau / (c * (double)gamma + 1.0);
}

vt_status vt_build_vocab(const int32_t* ids, int64_t n, int32_t V, int32_t K, int32_t* map,
                         int32_t* inv_map, void* ws, size_t ws_bytes, void* stream) {
    if (n < 0 || n >= ((int64_t)1 << 32) || V < 1 || K < 1 || K > V || !map || !inv_map || (n > 0 && !ids))
        return VT_ERR_INVALID_ARG;
    if (!aligned(ids, 4)) return VT_ERR_INVALID_ARG;
    if (!hist_shape_ok(V)) return VT_ERR_UNSUPPORTED;
    vt_status st = check_ws(ws, ws_bytes, vt_workspace_bytes(VT_OP_BUILD_VOCAB, n, V, K, 0, 0, 0));
    if (st != VT_OK) return st;
    uint8_t* base = static_cast<uint8_t*>(ws);
    uint32_t* counts = reinterpret_cast<uint32_t*>(base + VT_CTRL_BYTES);
    uint8_t* inner = base + VT_CTRL_BYTES + align_up((size_t)V * 4, 256);
    cudaStream_t s = as_stream(stream);
    cudaError_t e = launch_histogram(ids, n, V, counts, 0, reinterpret_cast<Ctrl*>(base), inner, s);
    if (e != cudaSuccess) return from_cuda(e);
    return from_cuda(launch_select_topk(counts, V, K, map, inv_map, inner, s));
}

vt_status vt_build_vocab_host(const int32_t* ids_host, int64_t n, int32_t V, int32_t K,
                              int32_t* map, int32_t* inv_map, void* ws, size_t ws_bytes,
                              void* stream) {
    if (n < 0 || n >= ((int64_t)1 << 32) || V < 1 || K < 1 || K > V || !map || !inv_map ||
        (n > 0 && !ids_host))
        return VT_ERR_INVALID_ARG;
    if (!hist_shape_ok(V)) return VT_ERR_UNSUPPORTED;
    vt_status st = check_ws(ws, ws_bytes, vt_workspace_bytes(VT_OP_BUILD_VOCAB_HOST, n, V, K, 0, 0, 0));
    if (st != VT_OK) return st;
    uint8_t* base = static_cast<uint8_t*>(ws);
    Ctrl* ctrl = reinterpret_cast<Ctrl*>(base);
    uint32_t* counts = reinterpret_cast<uint32_t*>(base + VT_CTRL_BYTES);
    uint8_t* inner = base + VT_CTRL_BYTES + align_up((size_t)V * 4, 256);
    const size_t dev_part = vt_workspace_bytes(VT_OP_BUILD_VOCAB, n, V, K, 0, 0, 0);
    const int64_t chunk = n < kHostChunkIds ? (n > 0 ? n : 1) : kHostChunkIds;
    int32_t* stage[2];
    stage[0] = reinterpret_cast<int32_t*>(base + align_up(dev_part, 256));
    stage[1] = reinterpret_cast<int32_t*>(reinterpret_cast<uint8_t*>(stage[0]) + align_up((size_t)chunk * 4, 256));
    cudaStream_t s = as_stream(stream);
    // Copies run on a second stream so chunk i+1 arrives while chunk i is counted; events order
    // "copy done -> count" and "count done -> buffer may be overwritten".
    cudaStream_t copy_stream = nullptr;
    cudaEvent_t copied[2] = {nullptr, nullptr}, counted[2] = {nullptr, nullptr}, start = nullptr;
    cudaError_t e = cudaStreamCreateWithFlags(&copy_stream, cudaStreamNonBlocking);
    for (int i = 0; i < 2 && e == cudaSuccess; ++i) {
        e = cudaEventCreateWithFlags(&copied[i], cudaEventDisableTiming);
        if (e == cudaSuccess) e = cudaEventCreateWithFlags(&counted[i], cudaEventDisableTiming);
    }
    if (e == cudaSuccess) e = cudaEventCreateWithFlags(&start, cudaEventDisableTiming);
    if (e == cudaSuccess) e = cudaMemsetAsync(counts, 0, (size_t)V * 4, s);
    if (e == cudaSuccess) e = cudaEventRecord(start, s);
    if (e == cudaSuccess) e = cudaStreamWaitEvent(copy_stream, start, 0);   // staging free once prior work on s is done
    int64_t done = 0;
    for (int i = 0; done < n && e == cudaSuccess; ++i) {
        const int sl = i & 1;
        const int64_t m = (n - done < chunk) ? n - done : chunk;
        if (i >= 2) e = cudaStreamWaitEvent(copy_stream, counted[sl], 0);
        if (e == cudaSuccess)
            e = cudaMemcpyAsync(stage[sl], ids_host + done, (size_t)m * 4, cudaMemcpyHostToDevice, copy_stream);
        if (e == cudaSuccess) e = cudaEventRecord(copied[sl], copy_stream);
        if (e == cudaSuccess) e = cudaStreamWaitEvent(s, copied[sl], 0);
        if (e == cudaSuccess) e = launch_histogram(stage[sl], m, V, counts, 1, ctrl, inner, s);
        if (e == cudaSuccess) e = cudaEventRecord(counted[sl], s);
        done += m;
    }
    if (e == cudaSuccess) e = launch_select_topk(counts, V, K, map, inv_map, inner, s);
    for (int i = 0; i < 2; ++i) {
        if (copied[i]) cudaEventDestroy(copied[i]);
        if (counted[i]) cudaEventDestroy(counted[i]);
    }
    if (start) cudaEventDestroy(start);
    if (copy_stream) cudaStreamDestroy(copy_stream);    // deferred until its work completes
    return from_cuda(e);
}

vt_status vt_trim_head(const uint16_t* W_full, const int32_t* map, uint16_t* W_trim, int32_t V,
                       int32_t K, int32_t d, void* ws, void* stream) {
    if (!W_full || !map || !W_trim || V < 1 || K < 1 || d < 8 || (d & 7)) return VT_ERR_INVALID_ARG;
    if (!aligned(W_full, 16) || !aligned(W_trim, 16) || !aligned(map, 4)) return VT_ERR_INVALID_ARG;
    if (ws && !aligned(ws, 256)) return VT_ERR_WORKSPACE;
    return from_cuda(launch_gather_rows(W_full, map, W_trim, V, K, d, static_cast<Ctrl*>(ws),
                                        as_stream(stream)));
}

static vt_status draft_head_impl(const uint16_t* h, const uint16_t* W_trim, const int32_t* map,
                                 int32_t B, int32_t K, int32_t d, const float* temp, int32_t topk,
                                 const float* uniforms, int32_t* out_ids, float* out_logprobs,
                                 void* ws, size_t ws_bytes, void* stream, float* out_logits,
                                 float* out_lse, int overlap, const TreeArgs& tree = TreeArgs{}) {
    if (!h || !W_trim || !temp || !out_ids || !out_logprobs) return VT_ERR_INVALID_ARG;
    if (B < 1 || K < 1 || d < 8 || (d & 7) || topk < 1 || topk > VT_MAX_TOPK || topk > K)
        return VT_ERR_INVALID_ARG;
    if (!aligned(h, 16) || !aligned(W_trim, 16)) return VT_ERR_INVALID_ARG;
    if (!head_shape_ok(B, K, d, topk)) return VT_ERR_UNSUPPORTED;
    vt_status st = check_ws(ws, ws_bytes, vt_workspace_bytes(VT_OP_DRAFT_HEAD, 0, 0, K, d, B, topk));
    if (st != VT_OK) return st;
    uint8_t* base = static_cast<uint8_t*>(ws);
    HeadArgs a{h, W_trim, map, B, K, d, temp, topk, uniforms, out_ids, out_logprobs, out_logits, out_lse, overlap, tree};
    if (head_skinny_supported(B, d))
        return from_cuda(launch_head_skinny(a, reinterpret_cast<Ctrl*>(base), base + VT_CTRL_BYTES,
                                            as_stream(stream)));
    return from_cuda(launch_head_dense(a, reinterpret_cast<Ctrl*>(base), base + VT_CTRL_BYTES,
                                       as_stream(stream)));
}

vt_status vt_draft_head_debug(const uint16_t* h, const uint16_t* W_trim, const int32_t* map,
                              int32_t B, int32_t K, int32_t d, const float* temp, int32_t topk,
                              const float* uniforms, int32_t* out_ids, float* out_logprobs,
                              void* ws, size_t ws_bytes, void* stream, float* out_logits,
                              float* out_lse) {
    return draft_head_impl(h, W_trim, map, B, K, d, temp, topk, uniforms, out_ids, out_logprobs, ws, ws_bytes,
                           stream, out_logits, out_lse, 0);
}

vt_status vt_draft_head(const uint16_t* h, const uint16_t* W_trim, const int32_t* map, int32_t B,
                        int32_t K, int32_t d, const float* temp, int32_t topk,
                        const float* uniforms, int32_t* out_ids, float* out_logprobs, void* ws,
                        size_t ws_bytes, void* stream) {
    return draft_head_impl(h, W_trim, map, B, K, d, temp, topk, uniforms, out_ids, out_logprobs, ws, ws_bytes,
                           stream, nullptr, nullptr, 0);
}

vt_status vt_draft_head_overlapped(const uint16_t* h, const uint16_t* W_trim, const int32_t* map, int32_t B,
                                   int32_t K, int32_t d, const float* temp, int32_t topk,
                                   const float* uniforms, int32_t* out_ids, float* out_logprobs, void* ws,
                                   size_t ws_bytes, void* stream) {
    return draft_head_impl(h, W_trim, map, B, K, d, temp, topk, uniforms, out_ids, out_logprobs, ws, ws_bytes,
                           stream, nullptr, nullptr, 1);
}

vt_status vt_draft_head_expand(const uint16_t* h, const uint16_t* W_trim, const int32_t* map, int32_t B,
                               int32_t K, int32_t d, const float* temp, int32_t topk, const float* uniforms,
                               int32_t* out_ids, float* out_logprobs, const int32_t* frontier_nodes,
                               int32_t* pool_token, int32_t* pool_parent, float* pool_score, int32_t pool_base,
                               int32_t pool_capacity, int32_t n_front, int32_t* next_frontier, void* ws,
                               size_t ws_bytes, void* stream) {
    const vt_status st = check_tree_args(B, topk, frontier_nodes, pool_token, pool_parent, pool_score, pool_base,
                                         pool_capacity, n_front, next_frontier);
    if (st != VT_OK) return st;
    const TreeArgs t{frontier_nodes, pool_token, pool_parent, pool_score, pool_base, n_front, next_frontier};
    return draft_head_impl(h, W_trim, map, B, K, d, temp, topk, uniforms, out_ids, out_logprobs, ws, ws_bytes,
                           stream, nullptr, nullptr, 1, t);
}

// Device-side address of a host buffer the device can reach (page-locked memory), else nullptr.
static void* mapped_host(const void* p) {
    cudaPointerAttributes at{};
    if (cudaPointerGetAttributes(&at, p) != cudaSuccess) { cudaGetLastError(); return nullptr; }
    return at.type == cudaMemoryTypeHost ? at.devicePointer : nullptr;
}

vt_status vt_draft_head_host(const uint16_t* h_host, const uint16_t* W_trim, const int32_t* map,
                             int32_t B, int32_t K, int32_t d, const float* temp_host, int32_t topk,
                             const float* uniforms_host, int32_t* out_ids_host,
                             float* out_logprobs_host, void* ws, size_t ws_bytes, void* stream) {
    if (!h_host || !W_trim || !temp_host || !out_ids_host || !out_logprobs_host) return VT_ERR_INVALID_ARG;
    if (B < 1 || K < 1 || d < 8 || (d & 7) || topk < 1 || topk > VT_MAX_TOPK || topk > K)
        return VT_ERR_INVALID_ARG;
    if (!head_shape_ok(B, K, d, topk)) return VT_ERR_UNSUPPORTED;
    vt_status st = check_ws(ws, ws_bytes, vt_workspace_bytes(VT_OP_DRAFT_HEAD_HOST, 0, 0, K, d, B, topk));
    if (st != VT_OK) return st;
    uint8_t* base = static_cast<uint8_t*>(ws);
    const size_t head_part = VT_CTRL_BYTES + head_scratch(B, K, d, topk);
    const HostStage hs = host_stage(B, K, d, topk, head_part);
    cudaStream_t s = as_stream(stream);
    uint16_t* dh = reinterpret_cast<uint16_t*>(base + hs.off_h);
    float* dt = reinterpret_cast<float*>(base + hs.off_temp);
    float* du = reinterpret_cast<float*>(base + hs.off_u);
    int32_t* di = reinterpret_cast<int32_t*>(base + hs.off_ids);
    float* dl = reinterpret_cast<float*>(base + hs.off_lp);
    const size_t out_bytes = (size_t)B * (1 + topk) * 4;
    // Small buffers in page-locked host memory are used in place: the kernels read the B temperatures and
    // write the B * (1 + topk) results through the device's mapping of that memory, which saves three of
    // the five copies of a step.  Pageable buffers go through the workspace as before.
    int32_t* oi = static_cast<int32_t*>(mapped_host(out_ids_host));
    float* ol = static_cast<float*>(mapped_host(out_logprobs_host));
    const float* tp = static_cast<const float*>(mapped_host(temp_host));
    const bool out_in_place = oi && ol;
    cudaError_t e = cudaMemcpyAsync(dh, h_host, (size_t)B * d * 2, cudaMemcpyHostToDevice, s);
    if (e == cudaSuccess && !tp) e = cudaMemcpyAsync(dt, temp_host, (size_t)B * 4, cudaMemcpyHostToDevice, s);
    if (e == cudaSuccess && uniforms_host)
        e = cudaMemcpyAsync(du, uniforms_host, (size_t)B * K * 4, cudaMemcpyHostToDevice, s);
    if (e != cudaSuccess) return from_cuda(e);
    st = vt_draft_head(dh, W_trim, map, B, K, d, tp ? tp : dt, topk, uniforms_host ? du : nullptr,
                       out_in_place ? oi : di, out_in_place ? ol : dl, ws, head_part, stream);
    if (st != VT_OK || out_in_place) return st;
    e = cudaMemcpyAsync(out_ids_host, di, out_bytes, cudaMemcpyDeviceToHost, s);
    if (e == cudaSuccess) e = cudaMemcpyAsync(out_logprobs_host, dl, out_bytes, cudaMemcpyDeviceToHost, s);
    return from_cuda(e);
}

}  // extern "C"
