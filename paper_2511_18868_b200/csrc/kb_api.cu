// C ABI of libkb: context, argument validation, the call sequence of a whole
// bandit step (device-resident and host-buffer variants).
#include <stdarg.h>
#include <string.h>

#include <new>

#include "kb_internal.cuh"

kb_status kb_fail(kb_ctx* ctx, kb_status s, const char* fmt, ...) {
    if (ctx) {
        va_list ap;
        va_start(ap, fmt);
        vsnprintf(ctx->err, sizeof(ctx->err), fmt, ap);
        va_end(ap);
    }
    return s;
}

namespace {

__global__ void gather_rows_kernel(int N, int D, int K, const float* __restrict__ z, const int32_t* __restrict__ rows,
                                   float* __restrict__ c, int* __restrict__ dev_status) {
    kb_grid_dependency_wait();
    const int b = blockIdx.y, i = blockIdx.x;
    int r = rows[(size_t)b * K + i];
    float* dst = c + ((size_t)b * K + i) * D;
    if (r == -1) {                                                  // an unused cluster: out of every row's reach
        for (int d = threadIdx.x; d < D; d += blockDim.x) dst[d] = KB_UNUSED_CENTROID;
        return;
    }
    if (r < 0 || r >= N) { if (threadIdx.x == 0) atomicOr(dev_status, 4); return; }
    const float* src = z + ((size_t)b * N + r) * D;
    for (int d = threadIdx.x; d < D; d += blockDim.x) dst[d] = src[d];
}

size_t max_sz(size_t a, size_t b) { return a > b ? a : b; }

// Tolerance stop for a fit that runs as a loop of calls (no host read, no change to the kernels of the loop): after
// every update this kernel (one CTA per instance) measures the instance's total squared centroid shift against the
// copy it keeps of the previous centroids.  An instance whose shift has dropped to `tol` is DONE from then on: the
// update that got it there stays, every later update (and its counts) is undone by restoring the copy, so the
// remaining iterations recompute the same labels and the final assignment sees the centroids the instance stopped
// at -- the result of stopping, at the cost of the idle iterations.
// mode 0: before the loop (copy <- centroids, done <- 0); mode 1: after update number `it`; mode 2: n_iter out.
__global__ void __launch_bounds__(256) tol_gate_kernel(int mode, int it, int KD, int K, float tol, float* __restrict__ cent,
                                                       int32_t* __restrict__ counts, float* __restrict__ prev,
                                                       int32_t* __restrict__ prev_counts, int32_t* __restrict__ done,
                                                       int32_t* __restrict__ n_iter) {
    kb_grid_dependency_wait();
    __shared__ double s_red[8];
    __shared__ int s_frozen;
    const int b = blockIdx.x, tid = threadIdx.x;
    float* c = cent + (size_t)b * KD;
    float* p = prev + (size_t)b * KD;
    if (mode == 0) {
        for (int e = tid; e < KD; e += 256) p[e] = c[e];
        if (tid == 0) done[b] = 0;
        return;
    }
    if (mode == 2) {
        if (tid == 0 && n_iter) n_iter[b] = done[b] ? done[b] : it;
        return;
    }
    if (tid == 0) s_frozen = done[b];
    __syncthreads();
    const bool frozen = s_frozen != 0;
    if (frozen) {
        for (int e = tid; e < KD; e += 256) c[e] = p[e];
        if (counts) for (int j = tid; j < K; j += 256) counts[(size_t)b * K + j] = prev_counts[(size_t)b * K + j];
        return;
    }
    double moved = 0.0;
    for (int e = tid; e < KD; e += 256) {
        const float dlt = c[e] - p[e];
        moved += (double)dlt * (double)dlt;
        p[e] = c[e];
    }
    if (counts) for (int j = tid; j < K; j += 256) prev_counts[(size_t)b * K + j] = counts[(size_t)b * K + j];
    const double w = kb_warp_sum(moved);
    if ((tid & 31) == 0) s_red[tid >> 5] = w;
    __syncthreads();
    if (tid == 0) {
        double shift = 0.0;
        for (int q = 0; q < 8; ++q) shift += s_red[q];
        if (shift <= (double)tol) done[b] = it;
    }
}

size_t ws_need_tol(int B, int D, int K) {
    return kb_align256((size_t)B * K * D * sizeof(float)) + kb_align256((size_t)B * K * sizeof(int32_t)) +
           kb_align256((size_t)B * sizeof(int32_t));
}

// brackets the work one public call queues with a pair of events (when timing is on)
struct TimeScope {
    kb_ctx* ctx;
    int slot;
    TimeScope(kb_ctx* c, int cls) : ctx(c), slot(-1) {
        if (c && c->timing && c->ev_used < KB_EV_PAIRS) {
            slot = c->ev_used++;
            c->ev_class[slot] = (unsigned char)cls;
            cudaEventRecord(c->ev[2 * slot], c->stream);
        }
    }
    ~TimeScope() {
        if (slot >= 0) cudaEventRecord(ctx->ev[2 * slot + 1], ctx->stream);
    }
};

}  // namespace

// What a device status word means for the caller of a synchronising entry point.
kb_status kb_status_from_device_word(kb_ctx* ctx, int word, bool contract_bits_too) {
    if (word & (KB_STATUS_TIMEOUT_ASSIGN | KB_STATUS_TIMEOUT_FIT))
        return kb_fail(ctx, KB_ERR_TIMEOUT, "a bounded device-side wait expired (device status 0x%x)", word);
    if (contract_bits_too && (word & (KB_STATUS_BAD_LABEL | KB_STATUS_BAD_TARGET | KB_STATUS_BAD_INDEX)))
        return kb_fail(ctx, KB_ERR_INVALID_ARG, "a label, target or index on the device was out of range (device status 0x%x)",
                       word);
    return KB_OK;
}

kb_status kb_launch_init_centroids(kb_ctx* ctx, int B, int N, int D, int K, const float* z, const int32_t* rows,
                                   float* c) {
    if (B == 0 || K == 0) return KB_OK;
    kb_launch(gather_rows_kernel, dim3(K, B), 64, 0, ctx->stream, N, D, K, z, rows, c, ctx->dev_status);
    KB_LAUNCH_CHECK(ctx, "gather_rows_kernel");
    return KB_OK;
}

extern "C" {

const char* kb_status_string(kb_status s) {
    switch (s) {
        case KB_OK: return "KB_OK";
        case KB_ERR_INVALID_ARG: return "KB_ERR_INVALID_ARG";
        case KB_ERR_UNSUPPORTED: return "KB_ERR_UNSUPPORTED";
        case KB_ERR_WORKSPACE: return "KB_ERR_WORKSPACE";
        case KB_ERR_CUDA: return "KB_ERR_CUDA";
        case KB_ERR_TIMEOUT: return "KB_ERR_TIMEOUT";
        default: return "KB_ERR_UNKNOWN";
    }
}

kb_status kb_create(kb_ctx** out, int device, void* cuda_stream) {
    if (!out) return KB_ERR_INVALID_ARG;
    *out = nullptr;
    int count = 0;
    if (cudaGetDeviceCount(&count) != cudaSuccess || device < 0 || device >= count) return KB_ERR_CUDA;
    kb_ctx* ctx = new (std::nothrow) kb_ctx();
    if (!ctx) return KB_ERR_CUDA;
    memset(ctx, 0, sizeof(*ctx));
    ctx->device = device;
    ctx->stream = static_cast<cudaStream_t>(cuda_stream);
    ctx->tc_eps = 1.0f / 65536.0f;
    cudaError_t e = cudaSetDevice(device);
    if (e == cudaSuccess) e = cudaDeviceGetAttribute(&ctx->sm_count, cudaDevAttrMultiProcessorCount, device);
    if (e == cudaSuccess) e = cudaDeviceGetAttribute(&ctx->max_smem_optin, cudaDevAttrMaxSharedMemoryPerBlockOptin, device);
    if (e == cudaSuccess) e = cudaDeviceGetAttribute(&ctx->coop_launch, cudaDevAttrCooperativeLaunch, device);
    // the host-buffer step copies the inputs its last calls need on a stream of its own, beside the clustering
    if (e == cudaSuccess) e = cudaStreamCreateWithFlags(&ctx->copy_stream, cudaStreamNonBlocking);
    if (e == cudaSuccess) e = cudaEventCreateWithFlags(&ctx->ev_step_begin, cudaEventDisableTiming);
    if (e == cudaSuccess) e = cudaEventCreateWithFlags(&ctx->ev_late_inputs, cudaEventDisableTiming);
    if (e == cudaSuccess) e = cudaStreamCreateWithFlags(&ctx->early_stream, cudaStreamNonBlocking);
    if (e == cudaSuccess) e = cudaEventCreateWithFlags(&ctx->ev_prune_inputs, cudaEventDisableTiming);
    if (e == cudaSuccess) e = cudaEventCreateWithFlags(&ctx->ev_bound_done, cudaEventDisableTiming);
    if (e == cudaSuccess) e = cudaMalloc(&ctx->dev_status, 256);
    if (e == cudaSuccess) e = cudaMemset(ctx->dev_status, 0, 256);
    if (e != cudaSuccess) {
        if (ctx->dev_status) cudaFree(ctx->dev_status);
        if (ctx->ev_bound_done) cudaEventDestroy(ctx->ev_bound_done);
        if (ctx->ev_prune_inputs) cudaEventDestroy(ctx->ev_prune_inputs);
        if (ctx->early_stream) cudaStreamDestroy(ctx->early_stream);
        if (ctx->ev_late_inputs) cudaEventDestroy(ctx->ev_late_inputs);
        if (ctx->ev_step_begin) cudaEventDestroy(ctx->ev_step_begin);
        if (ctx->copy_stream) cudaStreamDestroy(ctx->copy_stream);
        delete ctx;
        return KB_ERR_CUDA;
    }
    *out = ctx;
    return KB_OK;
}

kb_status kb_timing_enable(kb_ctx* ctx, int on) {
    if (!ctx) return KB_ERR_INVALID_ARG;
    if (on && !ctx->ev) {
        ctx->ev = new (std::nothrow) cudaEvent_t[2 * KB_EV_PAIRS];
        ctx->ev_class = new (std::nothrow) unsigned char[KB_EV_PAIRS];
        if (!ctx->ev || !ctx->ev_class) return kb_fail(ctx, KB_ERR_CUDA, "kb_timing_enable: out of host memory");
        for (int i = 0; i < 2 * KB_EV_PAIRS; ++i) KB_CUDA(ctx, cudaEventCreate(&ctx->ev[i]));
    }
    ctx->timing = on != 0;
    ctx->ev_used = 0;
    return KB_OK;
}

kb_status kb_timing_read(kb_ctx* ctx, double* ms, int64_t* calls) {
    if (!ctx || !ms || !calls) return KB_ERR_INVALID_ARG;
    for (int i = 0; i < KB_T_COUNT; ++i) { ms[i] = 0.0; calls[i] = 0; }
    KB_CUDA(ctx, cudaStreamSynchronize(ctx->stream));
    for (int s = 0; s < ctx->ev_used; ++s) {
        float t = 0.f;
        KB_CUDA(ctx, cudaEventElapsedTime(&t, ctx->ev[2 * s], ctx->ev[2 * s + 1]));
        ms[ctx->ev_class[s]] += (double)t;
        calls[ctx->ev_class[s]]++;
    }
    ctx->ev_used = 0;
    return KB_OK;
}

kb_status kb_destroy(kb_ctx* ctx) {
    if (!ctx) return KB_OK;
    cudaSetDevice(ctx->device);
    if (ctx->ev) {
        for (int i = 0; i < 2 * KB_EV_PAIRS; ++i) cudaEventDestroy(ctx->ev[i]);
        delete[] ctx->ev;
        delete[] ctx->ev_class;
    }
    if (ctx->dev_status) cudaFree(ctx->dev_status);
    if (ctx->ev_bound_done) cudaEventDestroy(ctx->ev_bound_done);
    if (ctx->ev_prune_inputs) cudaEventDestroy(ctx->ev_prune_inputs);
    if (ctx->early_stream) cudaStreamDestroy(ctx->early_stream);
    if (ctx->ev_late_inputs) cudaEventDestroy(ctx->ev_late_inputs);
    if (ctx->ev_step_begin) cudaEventDestroy(ctx->ev_step_begin);
    if (ctx->copy_stream) cudaStreamDestroy(ctx->copy_stream);
    delete ctx;
    return KB_OK;
}

kb_status kb_set_stream(kb_ctx* ctx, void* cuda_stream) {
    if (!ctx) return KB_ERR_INVALID_ARG;
    ctx->stream = static_cast<cudaStream_t>(cuda_stream);
    return KB_OK;
}

// Scratch of the calls a fit makes; the pre-split image of Z that a fit keeps across its iterations
// lies behind it (the other calls never run inside a fit and may use that space).
static size_t fit_scratch_bytes(int B, int N, int D, int K) {
    size_t need = 256;
    need = max_sz(need, kb_ws_need_assign(B, N, D, K));
    need = max_sz(need, kb_ws_need_update(B, N, D, K));
    need = max_sz(need, kb_ws_need_fit_coop(B, N, D, K));
    return kb_align256(need) + 1024;
}

kb_status kb_workspace_bytes(int B, int N, int D, int K, int S, size_t* out) {
    if (!out || B < 0 || N < 0 || D < 0 || K < 0 || S < 0) return KB_ERR_INVALID_ARG;
    size_t need = 256;
    need = max_sz(need, kb_ws_need_normalize(B, N, D));
    need = max_sz(need, kb_ws_need_score(B, N, K, S));
    need = max_sz(need, kb_ws_need_sample(B));
    need = max_sz(need, kb_ws_need_seed(B, N, K));
    need = max_sz(need, kb_ws_need_topm(B, KB_TOP_M_MAX));
    need = max_sz(need, fit_scratch_bytes(B, N, D, K) + kb_ws_need_fit_acc(B, D, K) + kb_ws_need_zsplit(B, N, D, K) +
                            ws_need_tol(B, D, K));
    *out = need;
    return KB_OK;
}

kb_status kb_set_workspace(kb_ctx* ctx, void* dev_ptr, size_t bytes) {
    if (!ctx) return KB_ERR_INVALID_ARG;
    KB_REQUIRE(ctx, (dev_ptr != nullptr) == (bytes != 0), "kb_set_workspace: pointer and size disagree");
    KB_REQUIRE(ctx, ((uintptr_t)dev_ptr & 255) == 0, "kb_set_workspace: workspace must be 256-byte aligned");
    ctx->ws = static_cast<char*>(dev_ptr);
    ctx->ws_bytes = bytes;
    return KB_OK;
}

const char* kb_last_error(kb_ctx* ctx) { return ctx ? ctx->err : "no context"; }

kb_status kb_get_device_status(kb_ctx* ctx, int* out) {
    if (!ctx || !out) return KB_ERR_INVALID_ARG;
    KB_CUDA(ctx, cudaMemcpyAsync(out, ctx->dev_status, sizeof(int), cudaMemcpyDeviceToHost, ctx->stream));
    KB_CUDA(ctx, cudaStreamSynchronize(ctx->stream));
    return kb_status_from_device_word(ctx, *out, false);
}

kb_status kb_status_of_device_word(int word, int contract_bits_too) {
    return kb_status_from_device_word(nullptr, word, contract_bits_too != 0);
}

kb_status kb_debug_wait_limit(kb_ctx* ctx, unsigned polls, int leave_one_out) {
    if (!ctx) return KB_ERR_INVALID_ARG;
    ctx->dbg_wait_limit = polls;
    ctx->dbg_skip_arrival = leave_one_out != 0;
    return KB_OK;
}

namespace {
__global__ void __launch_bounds__(256) count_nonfinite_kernel(const float* __restrict__ x, size_t n,
                                                              unsigned long long* __restrict__ out) {
    unsigned long long c = 0;
    for (size_t i = (size_t)blockIdx.x * blockDim.x + threadIdx.x; i < n; i += (size_t)gridDim.x * blockDim.x) {
        const unsigned u = __float_as_uint(__ldg(x + i));
        c += (u & 0x7f800000u) == 0x7f800000u;               // exponent all ones: NaN or infinity
    }
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) c += __shfl_xor_sync(0xffffffffu, c, o);
    if ((threadIdx.x & 31) == 0 && c) atomicAdd(out, c);
}
}  // namespace

kb_status kb_debug_count_nonfinite(kb_ctx* ctx, const float* x, size_t n, uint64_t* out) {
    if (!ctx || !out || (n > 0 && !x)) return KB_ERR_INVALID_ARG;
    *out = 0;
    if (n == 0) return KB_OK;
    // a 64-bit counter in the spare words behind the status word (the context owns 256 bytes there)
    unsigned long long* cnt = reinterpret_cast<unsigned long long*>(ctx->dev_status + 48);
    KB_MEMSET(ctx, cnt, 0, sizeof(unsigned long long));
    size_t blocks = (n + 255) / 256;
    const size_t cap = (size_t)ctx->sm_count * 8;
    if (blocks > cap) blocks = cap;
    kb_launch(count_nonfinite_kernel, (unsigned)blocks, 256, 0, ctx->stream, x, n, cnt);
    KB_LAUNCH_CHECK(ctx, "count_nonfinite_kernel");
    unsigned long long host = 0;
    KB_CUDA(ctx, cudaMemcpyAsync(&host, cnt, sizeof(host), cudaMemcpyDeviceToHost, ctx->stream));
    KB_CUDA(ctx, cudaStreamSynchronize(ctx->stream));
    *out = host;
    return KB_OK;
}

kb_status kb_clear_device_status(kb_ctx* ctx) {
    if (!ctx) return KB_ERR_INVALID_ARG;
    KB_MEMSET(ctx, ctx->dev_status, 0, sizeof(int));
    return KB_OK;
}

kb_status kb_get_launch_count(kb_ctx* ctx, uint64_t* kernels, uint64_t* memsets) {
    if (!ctx || !kernels) return KB_ERR_INVALID_ARG;
    *kernels = ctx->launches;
    if (memsets) *memsets = ctx->memsets;
    return KB_OK;
}

#define KB_COMMON(ctx, B, N)                                                                   \
    do {                                                                                       \
        if (!(ctx)) return KB_ERR_INVALID_ARG;                                                 \
        KB_REQUIRE(ctx, (B) >= 0 && (N) >= 0, "negative size");                                \
        if ((B) > 65535) return kb_fail(ctx, KB_ERR_UNSUPPORTED, "B = %d exceeds 65535", (B)); \
    } while (0)

kb_status kb_normalize(kb_ctx* ctx, int B, int N, int D, const float* x, float* z, float* mean, float* scale) {
    KB_COMMON(ctx, B, N);
    KB_REQUIRE(ctx, D >= 1, "kb_normalize: D must be >= 1");
    if ((size_t)B * N > 0) KB_REQUIRE(ctx, x && z, "kb_normalize: x and z are required");
    if (D % 4 == 0)
        KB_REQUIRE(ctx, (((uintptr_t)x | (uintptr_t)z) & 15) == 0, "kb_normalize: x and z must be 16-byte aligned");
    TimeScope ts__(ctx, KB_T_NORMALIZE);
    return kb_launch_normalize(ctx, B, N, D, x, z, mean, scale);
}

kb_status kb_prune(kb_ctx* ctx, int B, int N, int S, int K, int R, const float* flops, const float* bytes,
                   const float* peak_flops, const float* peak_bw, const float* t_incumbent, const float* t_cur,
                   const int32_t* labels, const float* hsig, const int32_t* target, float theta_sat, uint32_t* keep,
                   uint32_t* kept_count, float* bound) {
    KB_COMMON(ctx, B, N);
    KB_REQUIRE(ctx, S >= 1, "kb_prune: S must be >= 1");
    if (S > 32) return kb_fail(ctx, KB_ERR_UNSUPPORTED, "kb_prune: S = %d exceeds 32 (keep bits are 32 wide)", S);
    KB_REQUIRE(ctx, peak_flops && peak_bw, "kb_prune: the ceilings table is required");
    if (B > 0) KB_REQUIRE(ctx, t_incumbent, "kb_prune: t_incumbent is required");
    if ((size_t)B * N > 0) KB_REQUIRE(ctx, flops && bytes && keep, "kb_prune: flops, bytes and keep are required");
    const int nsat = (labels != nullptr) + (hsig != nullptr) + (target != nullptr);
    KB_REQUIRE(ctx, nsat == 0 || nsat == 3, "kb_prune: labels, hsig and target must be given together");
    if (nsat == 3) KB_REQUIRE(ctx, K >= 1 && R >= 1, "kb_prune: K and R must be >= 1 with the saturation mask");
    if (bound) KB_REQUIRE(ctx, t_cur, "kb_prune: bound needs t_cur");
    TimeScope ts__(ctx, KB_T_PRUNE);
    return kb_launch_prune(ctx, B, N, S, K, R, flops, bytes, peak_flops, peak_bw, t_incumbent, t_cur, labels, hsig,
                           target, theta_sat, keep, kept_count, bound);
}

kb_status kb_cluster_assign(kb_ctx* ctx, int B, int N, int D, int K, const float* z, const float* centroids,
                            int32_t* labels, float* dist2, float* inertia, int32_t* rep) {
    KB_COMMON(ctx, B, N);
    KB_REQUIRE(ctx, D >= 1 && K >= 1, "kb_cluster_assign: D and K must be >= 1");
    if (B > 0) KB_REQUIRE(ctx, centroids, "kb_cluster_assign: centroids are required");
    if ((size_t)B * N > 0) KB_REQUIRE(ctx, z && labels, "kb_cluster_assign: z and labels are required");
    if (D % 4 == 0)
        KB_REQUIRE(ctx, (((uintptr_t)z | (uintptr_t)centroids) & 15) == 0,
                   "kb_cluster_assign: z and centroids must be 16-byte aligned");
    TimeScope ts__(ctx, KB_T_ASSIGN);
    return kb_launch_assign(ctx, B, N, D, K, z, centroids, labels, dist2, inertia, rep);
}

kb_status kb_set_assign_options(kb_ctx* ctx, int path, float tc_eps) {
    if (!ctx) return KB_ERR_INVALID_ARG;
    KB_REQUIRE(ctx, path >= 0 && path <= 3, "kb_set_assign_options: path must be 0, 1, 2 or 3");
    ctx->assign_path = path;
    ctx->tc_eps = tc_eps > 0.f ? tc_eps : 1.0f / 65536.0f;
    return KB_OK;
}

kb_status kb_get_assign_path(kb_ctx* ctx, int* out) {
    if (!ctx || !out) return KB_ERR_INVALID_ARG;
    *out = ctx->last_assign_path;
    return KB_OK;
}

kb_status kb_get_assign_presplit(kb_ctx* ctx, int* out) {
    if (!ctx || !out) return KB_ERR_INVALID_ARG;
    *out = ctx->last_assign_presplit;
    return KB_OK;
}

kb_status kb_assign_tc_probe(kb_ctx* ctx, int B, int N, int D, int K, const float* z, const float* centroids,
                             int32_t* labels, float* approx_dist2, int32_t* flagged) {
    KB_COMMON(ctx, B, N);
    KB_REQUIRE(ctx, D >= 1 && K >= 1, "kb_assign_tc_probe: D and K must be >= 1");
    KB_REQUIRE(ctx, z && centroids && labels, "kb_assign_tc_probe: z, centroids and labels are required");
    if (!kb_assign_tc_supported(ctx, B, D, K))
        return kb_fail(ctx, KB_ERR_UNSUPPORTED, "kb_assign_tc_probe: needs D %% 32 == 0, D <= 128, K <= 8192");
    if (B == 0 || N == 0) return KB_OK;
    const size_t off = kb_ws_need_assign(B, N, D, K) - kb_ws_need_assign_tc(B, N, D, K);
    if (ctx->ws_bytes < kb_ws_need_assign(B, N, D, K))
        return kb_fail(ctx, KB_ERR_WORKSPACE, "kb_assign_tc_probe needs %zu bytes of workspace",
                       kb_ws_need_assign(B, N, D, K));
    TimeScope ts__(ctx, KB_T_ASSIGN);
    return kb_launch_assign_tc(ctx, ctx->ws + off, B, N, D, K, z, centroids, labels, approx_dist2, flagged, ctx->tc_eps);
}

kb_status kb_cluster_update(kb_ctx* ctx, int B, int N, int D, int K, const float* z, const int32_t* labels,
                            float* centroids, int32_t* counts) {
    KB_COMMON(ctx, B, N);
    KB_REQUIRE(ctx, D >= 1 && K >= 1, "kb_cluster_update: D and K must be >= 1");
    if (B > 0) KB_REQUIRE(ctx, centroids, "kb_cluster_update: centroids are required");
    if ((size_t)B * N > 0) KB_REQUIRE(ctx, z && labels, "kb_cluster_update: z and labels are required");
    if (D % 4 == 0) KB_REQUIRE(ctx, ((uintptr_t)z & 15) == 0, "kb_cluster_update: z must be 16-byte aligned");
    TimeScope ts__(ctx, KB_T_UPDATE);
    return kb_launch_update(ctx, B, N, D, K, z, labels, centroids, counts);
}

kb_status kb_score_select(kb_ctx* ctx, int B, int N, int K, int S, kb_score_params p, const int32_t* labels,
                          const float* dist2, const int32_t* pulls, const float* reward_sum, const uint32_t* keep,
                          const float* bound, const int32_t* t, float* cl_pulls, float* cl_mean, float* cl_index,
                          float* arm_index, int32_t* best_arm, float* best_val, int32_t* best_cluster_arm) {
    KB_COMMON(ctx, B, N);
    KB_REQUIRE(ctx, K >= 1 && S >= 1, "kb_score_select: K and S must be >= 1");
    if (S > 32) return kb_fail(ctx, KB_ERR_UNSUPPORTED, "kb_score_select: S = %d exceeds 32", S);
    if ((long long)N * S > 0x7fffffffLL)
        return kb_fail(ctx, KB_ERR_UNSUPPORTED, "kb_score_select: N*S exceeds the 31-bit arm index");
    KB_REQUIRE(ctx, p.prior_pulls > 0.f, "kb_score_select: prior_pulls must be positive");
    if (B > 0)
        KB_REQUIRE(ctx, t && cl_pulls && cl_mean && cl_index && best_arm && best_val && best_cluster_arm,
                   "kb_score_select: t and the per-cluster / per-instance outputs are required");
    if ((size_t)B * N > 0) {
        KB_REQUIRE(ctx, labels && pulls && reward_sum, "kb_score_select: labels, pulls and reward_sum are required");
        KB_REQUIRE(ctx, p.lipschitz_L == 0.f || dist2, "kb_score_select: dist2 is required when L != 0");
        KB_REQUIRE(ctx, !p.cap_with_bound || bound, "kb_score_select: cap_with_bound needs bound");
    }
    TimeScope ts__(ctx, KB_T_SCORE);
    return kb_launch_score(ctx, B, N, K, S, p, labels, dist2, pulls, reward_sum, keep, bound, t, cl_pulls, cl_mean,
                           cl_index, arm_index, best_arm, best_val, best_cluster_arm);
}

kb_status kb_sample_member(kb_ctx* ctx, int B, int N, int K, int S, int R, const int32_t* labels,
                           const int32_t* cluster_arm, const float* h_cand, const int32_t* target, float theta_sat,
                           uint64_t seed, const int32_t* t, int32_t* member, float* member_val) {
    KB_COMMON(ctx, B, N);
    KB_REQUIRE(ctx, K >= 1 && S >= 1 && R >= 1, "kb_sample_member: K, S and R must be >= 1");
    if ((long long)K * S > 0x7fffffffLL)
        return kb_fail(ctx, KB_ERR_UNSUPPORTED, "kb_sample_member: K*S exceeds the 31-bit pair index");
    if (B > 0)
        KB_REQUIRE(ctx, cluster_arm && target && t && member,
                   "kb_sample_member: cluster_arm, target, t and member are required");
    if ((size_t)B * N > 0) KB_REQUIRE(ctx, labels && h_cand, "kb_sample_member: labels and h_cand are required");
    TimeScope ts__(ctx, KB_T_SAMPLE);
    return kb_launch_sample_member(ctx, B, N, K, S, R, labels, cluster_arm, h_cand, target, theta_sat, seed, t, member,
                                   member_val);
}

kb_status kb_best_restart(kb_ctx* ctx, int G, int n_init, const float* inertia, int32_t* best) {
    if (!ctx) return KB_ERR_INVALID_ARG;
    KB_REQUIRE(ctx, G >= 0 && n_init >= 1, "kb_best_restart: G must be >= 0 and n_init >= 1");
    if (G > 0) KB_REQUIRE(ctx, inertia && best, "kb_best_restart: inertia and best are required");
    TimeScope ts__(ctx, KB_T_INIT);
    return kb_launch_best_restart(ctx, G, n_init, inertia, best);
}

kb_status kb_select_top_m(kb_ctx* ctx, int B, int N, int S, int M, const float* arm_index, int32_t* top_arm,
                          float* top_val) {
    KB_COMMON(ctx, B, N);
    KB_REQUIRE(ctx, S >= 1 && M >= 0, "kb_select_top_m: S must be >= 1 and M >= 0");
    if (M > KB_TOP_M_MAX) return kb_fail(ctx, KB_ERR_UNSUPPORTED, "kb_select_top_m: M = %d exceeds %d", M, KB_TOP_M_MAX);
    if ((long long)N * S > 0x7fffffffLL)
        return kb_fail(ctx, KB_ERR_UNSUPPORTED, "kb_select_top_m: N*S exceeds the 31-bit arm index");
    if (B > 0 && M > 0) KB_REQUIRE(ctx, top_arm, "kb_select_top_m: top_arm is required");
    if ((size_t)B * N > 0 && M > 0) KB_REQUIRE(ctx, arm_index, "kb_select_top_m: arm_index is required");
    TimeScope ts__(ctx, KB_T_SCORE);
    return kb_launch_top_m(ctx, B, N * S, M, arm_index, top_arm, top_val);
}

kb_status kb_cluster_radius(kb_ctx* ctx, int B, int N, int K, const int32_t* labels, const float* dist2, float* radius) {
    KB_COMMON(ctx, B, N);
    KB_REQUIRE(ctx, K >= 1, "kb_cluster_radius: K must be >= 1");
    if (B > 0) KB_REQUIRE(ctx, radius, "kb_cluster_radius: radius is required");
    if ((size_t)B * N > 0) KB_REQUIRE(ctx, labels && dist2, "kb_cluster_radius: labels and dist2 are required");
    TimeScope ts__(ctx, KB_T_SAMPLE);
    return kb_launch_cluster_radius(ctx, B, N, K, labels, dist2, radius);
}

kb_status kb_seed_kmeanspp(kb_ctx* ctx, int B, int N, int D, int K, const float* z, uint64_t seed, int32_t* rows) {
    KB_COMMON(ctx, B, N);
    KB_REQUIRE(ctx, D >= 1 && K >= 1, "kb_seed_kmeanspp: D and K must be >= 1");
    if (B > 0) {
        KB_REQUIRE(ctx, N >= 1, "kb_seed_kmeanspp: needs at least one row to draw from");
        KB_REQUIRE(ctx, z && rows, "kb_seed_kmeanspp: z and rows are required");
    }
    TimeScope ts__(ctx, KB_T_INIT);
    return kb_launch_seed_kmeanspp(ctx, B, N, D, K, z, seed, rows);
}

kb_status kb_select_pair(kb_ctx* ctx, int B, int K, int S, int R, float c, const float* cl_pulls, const float* cl_mean,
                         const int32_t* t, const float* hsig, const int32_t* target, float theta_sat, float* cl_index,
                         int32_t* pair) {
    KB_COMMON(ctx, B, 0);
    KB_REQUIRE(ctx, K >= 1 && S >= 1 && R >= 1, "kb_select_pair: K, S and R must be >= 1");
    if ((long long)K * S > 0x7fffffffLL) return kb_fail(ctx, KB_ERR_UNSUPPORTED, "kb_select_pair: K*S exceeds 31 bits");
    if (B > 0) {
        KB_REQUIRE(ctx, cl_pulls && cl_mean && t && pair, "kb_select_pair: cl_pulls, cl_mean, t and pair are required");
        KB_REQUIRE(ctx, !hsig || target, "kb_select_pair: the saturation mask needs target");
    }
    TimeScope ts__(ctx, KB_T_SCORE);
    return kb_launch_select_pair(ctx, B, K, S, R, c, cl_pulls, cl_mean, t, hsig, target, theta_sat, cl_index, pair);
}

kb_status kb_record_outcome(kb_ctx* ctx, int B, int N, int K, int S, int failures_count, const int32_t* member,
                            const int32_t* cluster_arm, const float* t_cur, const float* t_new,
                            const int32_t* verified, int32_t* pulls, float* reward_sum, int32_t* t, float* reward,
                            float* cl_pulls, float* cl_mean) {
    KB_COMMON(ctx, B, N);
    KB_REQUIRE(ctx, S >= 1 && K >= 1, "kb_record_outcome: K and S must be >= 1");
    KB_REQUIRE(ctx, (cl_pulls != nullptr) == (cl_mean != nullptr), "kb_record_outcome: cl_pulls and cl_mean go together");
    if (B > 0) {
        KB_REQUIRE(ctx, member && cluster_arm && t_new && t, "kb_record_outcome: member, cluster_arm, t_new and t are required");
        if (N > 0) KB_REQUIRE(ctx, t_cur && pulls && reward_sum, "kb_record_outcome: t_cur, pulls and reward_sum are required");
    }
    TimeScope ts__(ctx, KB_T_SAMPLE);
    return kb_launch_record_outcome(ctx, B, N, K, S, failures_count, member, cluster_arm, t_cur, t_new, verified, pulls,
                                    reward_sum, t, reward, cl_pulls, cl_mean);
}

kb_status kb_append_candidate(kb_ctx* ctx, int B, int N_cap, int D, int S, int R, const int32_t* verified,
                              const int32_t* parent, const float* x_new, const float* t_new, const float* flops_new,
                              const float* bytes_new, const float* h_new, int32_t* n_active, float* x, float* t_cur,
                              float* flops, float* bytes, float* h_cand, int32_t* labels, float* dist2, int32_t* pulls,
                              float* reward_sum, float* t_incumbent, int32_t* appended) {
    KB_COMMON(ctx, B, N_cap);
    KB_REQUIRE(ctx, D >= 1 && S >= 1 && R >= 1, "kb_append_candidate: D, S and R must be >= 1");
    if (B > 0) {
        KB_REQUIRE(ctx, parent && x_new && t_new && n_active, "kb_append_candidate: parent, x_new, t_new and n_active are required");
        KB_REQUIRE(ctx, N_cap == 0 || (x && t_cur && labels && pulls && reward_sum),
                   "kb_append_candidate: x, t_cur, labels, pulls and reward_sum are required");
        KB_REQUIRE(ctx, (flops != nullptr) == (flops_new != nullptr) && (bytes != nullptr) == (bytes_new != nullptr) &&
                            (h_cand != nullptr) == (h_new != nullptr),
                   "kb_append_candidate: flops, bytes and h_cand each go with their new row");
    }
    TimeScope ts__(ctx, KB_T_SAMPLE);
    return kb_launch_append_candidate(ctx, B, N_cap, D, S, R, verified, parent, x_new, t_new, flops_new, bytes_new, h_new,
                                      n_active, x, t_cur, flops, bytes, h_cand, labels, dist2, pulls, reward_sum, t_incumbent,
                                      appended);
}

kb_status kb_recluster_due(kb_ctx* ctx, int B, int tau, int K, const int32_t* t, const int32_t* n_active, int32_t* due,
                           int32_t* any_due) {
    KB_COMMON(ctx, B, 0);
    KB_REQUIRE(ctx, tau >= 1 && K >= 1, "kb_recluster_due: tau and K must be >= 1");
    if (B > 0) KB_REQUIRE(ctx, t && n_active && due, "kb_recluster_due: t, n_active and due are required");
    TimeScope ts__(ctx, KB_T_SAMPLE);
    return kb_launch_recluster_due(ctx, B, tau, K, t, n_active, due, any_due);
}

kb_status kb_signatures_from_reps(kb_ctx* ctx, int B, int N, int K, int R, const int32_t* rep, const float* h_cand,
                                  const int32_t* run_mask, float* hsig) {
    KB_COMMON(ctx, B, N);
    KB_REQUIRE(ctx, K >= 1 && R >= 1, "kb_signatures_from_reps: K and R must be >= 1");
    if (B > 0) KB_REQUIRE(ctx, rep && hsig && (N == 0 || h_cand), "kb_signatures_from_reps: rep, h_cand and hsig are required");
    TimeScope ts__(ctx, KB_T_SAMPLE);
    return kb_launch_signatures_from_reps(ctx, B, N, K, R, rep, h_cand, run_mask, hsig);
}

kb_status kb_init_centroids(kb_ctx* ctx, int B, int N, int D, int K, const float* z, const int32_t* rows,
                            float* centroids) {
    KB_COMMON(ctx, B, N);
    KB_REQUIRE(ctx, D >= 1 && K >= 1, "kb_init_centroids: D and K must be >= 1");
    if (B > 0) {
        KB_REQUIRE(ctx, N >= 1, "kb_init_centroids: needs at least one row to copy from");
        KB_REQUIRE(ctx, z && rows && centroids, "kb_init_centroids: z, rows and centroids are required");
    }
    TimeScope ts__(ctx, KB_T_INIT);
    return kb_launch_init_centroids(ctx, B, N, D, K, z, rows, centroids);
}

static kb_status fit_impl(kb_ctx* ctx, int B, int N, int D, int K, int iters, float tol, const float* z, float* centroids,
                          int32_t* labels, float* dist2, float* inertia, int32_t* rep, int32_t* counts, int32_t* n_iter);

kb_status kb_cluster_fit(kb_ctx* ctx, int B, int N, int D, int K, int iters, const float* z, float* centroids,
                         int32_t* labels, float* dist2, float* inertia, int32_t* rep, int32_t* counts) {
    return fit_impl(ctx, B, N, D, K, iters, -1.f, z, centroids, labels, dist2, inertia, rep, counts, nullptr);
}

kb_status kb_cluster_fit_tol(kb_ctx* ctx, int B, int N, int D, int K, int max_iter, float tol, const float* z,
                             float* centroids, int32_t* labels, float* dist2, float* inertia, int32_t* rep,
                             int32_t* counts, int32_t* n_iter) {
    if (!ctx) return KB_ERR_INVALID_ARG;
    KB_REQUIRE(ctx, tol >= 0.f, "kb_cluster_fit_tol: tol must be >= 0");
    if (B > 0) KB_REQUIRE(ctx, n_iter, "kb_cluster_fit_tol: n_iter is required");
    return fit_impl(ctx, B, N, D, K, max_iter, tol, z, centroids, labels, dist2, inertia, rep, counts, n_iter);
}

// tol < 0: the plain loop of `iters` iterations; else the tolerance stop (n_iter out)
static kb_status fit_impl(kb_ctx* ctx, int B, int N, int D, int K, int iters, float tol, const float* z, float* centroids,
                          int32_t* labels, float* dist2, float* inertia, int32_t* rep, int32_t* counts, int32_t* n_iter) {
    KB_COMMON(ctx, B, N);
    KB_REQUIRE(ctx, iters >= 0, "kb_cluster_fit: iters must be >= 0");
    const bool stop = tol >= 0.f;
    if (ctx->assign_path == 0 && kb_fit_fused_eligible(ctx, B, N, D, K) && z && centroids && labels &&
        (((uintptr_t)z | (uintptr_t)centroids) & 15) == 0) {
        // small instances: the whole loop in one launch, one CTA per instance
        KB_REQUIRE(ctx, D >= 1 && K >= 1, "kb_cluster_fit: D and K must be >= 1");
        TimeScope ts__(ctx, KB_T_FIT);
        return kb_launch_fit_fused(ctx, B, N, D, K, iters, z, nullptr, nullptr, nullptr, centroids, labels, dist2, inertia,
                                   rep, counts, nullptr, nullptr, tol, n_iter);
    }
    if (!stop && ctx->assign_path == 0 && !kb_assign_tc_eligible(ctx, B, N, D, K) && kb_fit_coop_eligible(ctx, B, N, D, K) && z &&
        centroids && labels && (((uintptr_t)z | (uintptr_t)centroids) & 15) == 0) {
        // one mid-sized instance: the whole loop in one cooperative launch, the rows resident on chip
        TimeScope ts__(ctx, KB_T_FIT);
        return kb_launch_fit_coop(ctx, N, D, K, iters, z, nullptr, nullptr, nullptr, centroids, labels, dist2, inertia, rep,
                                  counts);
    }
    // Tensor-core assignments of the same matrix, several times over: split Z into its fp16 pieces once and let
    // every assignment multiply out of that image (kept behind the scratch of the calls below).
    // Behind the scratch of the calls below: the accumulators of the loop's updates, then the image.
    kb_status s = KB_OK;
    const size_t aoff = fit_scratch_bytes(B, N, D, K), aneed = kb_ws_need_fit_acc(B, D, K);
    const size_t zneed = kb_ws_need_zsplit(B, N, D, K), zoff = aoff + aneed;
    const bool tensor = N > 0 && z && ctx->assign_path != 1 &&
                        (ctx->assign_path >= 2 ? kb_assign_tc_supported(ctx, B, D, K) : kb_assign_tc_eligible(ctx, B, N, D, K));
    if (tensor && iters >= 2 && zneed > 0 && ctx->ws_bytes >= zoff + zneed) {
        TimeScope ts__(ctx, KB_T_PREP);
        s = kb_zsplit_prepare(ctx, ctx->ws + zoff, B, N, D, K, z);
    }
    if (tensor && iters >= 1 && ctx->ws_bytes >= aoff + aneed) {
        // every assignment of the loop clears these in its fix-up kernel, the update that follows adds into them
        ctx->fit_acc = ctx->ws + aoff;
        ctx->fit_acc_bytes = aneed;
        ctx->fit_acc_clean = 0;
    }
    // tolerance stop: a gate kernel after every update (see tol_gate_kernel); its copies lie behind everything else
    const size_t toff = zoff + zneed;
    float* g_prev = nullptr;
    int32_t *g_counts = nullptr, *g_done = nullptr;
    if (stop && B > 0 && s == KB_OK) {
        KB_REQUIRE(ctx, D >= 1 && K >= 1 && centroids, "kb_cluster_fit_tol: D, K >= 1 and centroids are required");
        if (ctx->ws_bytes < toff + ws_need_tol(B, D, K)) {
            ctx->fit_acc = nullptr;
            kb_zsplit_forget(ctx);
            return kb_fail(ctx, KB_ERR_WORKSPACE, "kb_cluster_fit_tol needs %zu bytes of workspace", toff + ws_need_tol(B, D, K));
        }
        g_prev = reinterpret_cast<float*>(ctx->ws + toff);
        g_counts = reinterpret_cast<int32_t*>(ctx->ws + toff + kb_align256((size_t)B * K * D * sizeof(float)));
        g_done = reinterpret_cast<int32_t*>(reinterpret_cast<char*>(g_counts) + kb_align256((size_t)B * K * sizeof(int32_t)));
        kb_launch(tol_gate_kernel, B, 256, 0, ctx->stream, 0, 0, K * D, K, tol, centroids, counts, g_prev, g_counts, g_done, n_iter);
        if (cudaGetLastError() != cudaSuccess) s = kb_fail(ctx, KB_ERR_CUDA, "launch of tol_gate_kernel failed");
        else ctx->launches++;
    }
    for (int it = 0; it < iters && s == KB_OK; ++it) {
        s = kb_cluster_assign(ctx, B, N, D, K, z, centroids, labels, nullptr, nullptr, nullptr);
        if (s == KB_OK) s = kb_cluster_update(ctx, B, N, D, K, z, labels, centroids, counts);
        if (s == KB_OK && g_prev) {
            kb_launch(tol_gate_kernel, B, 256, 0, ctx->stream, 1, it + 1, K * D, K, tol, centroids, counts, g_prev, g_counts, g_done,
                      n_iter);
            if (cudaGetLastError() != cudaSuccess) s = kb_fail(ctx, KB_ERR_CUDA, "launch of tol_gate_kernel failed");
            else ctx->launches++;
        }
    }
    if (s == KB_OK) s = kb_cluster_assign(ctx, B, N, D, K, z, centroids, labels, dist2, inertia, rep);
    if (s == KB_OK && g_prev) {
        kb_launch(tol_gate_kernel, B, 256, 0, ctx->stream, 2, iters, K * D, K, tol, centroids, counts, g_prev, g_counts, g_done, n_iter);
        if (cudaGetLastError() != cudaSuccess) s = kb_fail(ctx, KB_ERR_CUDA, "launch of tol_gate_kernel failed");
        else ctx->launches++;
    }
    ctx->fit_acc = nullptr;
    kb_zsplit_forget(ctx);
    return s;
}

// normalise, initial centroids, Lloyd loop: three calls, or one launch for small instances
static kb_status step_cluster(kb_ctx* ctx, const kb_step_args* a) {
    if (ctx->assign_path == 0 && a->iters >= 0 && kb_fit_fused_eligible(ctx, a->B, a->N, a->D, a->K) && a->x && a->z &&
        a->init_rows && a->centroids && a->labels &&
        (((uintptr_t)a->x | (uintptr_t)a->z | (uintptr_t)a->centroids) & 15) == 0) {
        // at most 512 rows per instance: one CTA takes its instance from raw features to labels
        TimeScope ts__(ctx, KB_T_FIT);
        return kb_launch_fit_fused(ctx, a->B, a->N, a->D, a->K, a->iters, nullptr, a->x, a->z, a->init_rows, a->centroids,
                                   a->labels, a->dist2, a->inertia, a->rep, a->counts, a->n_active, a->run_mask);
    }
    if (a->n_active || a->run_mask)
        return kb_fail(ctx, KB_ERR_UNSUPPORTED, "n_active / run_mask need instances that cluster as one CTA each: at most "
                                                 "512 rows, D in {16, 32, 64}, 16-byte aligned x, z, centroids");
    if (ctx->assign_path == 0 && a->iters >= 0 && !kb_assign_tc_eligible(ctx, a->B, a->N, a->D, a->K) &&
        kb_fit_coop_eligible(ctx, a->B, a->N, a->D, a->K) && a->x && a->z && a->init_rows && a->centroids && a->labels &&
        (((uintptr_t)a->x | (uintptr_t)a->z | (uintptr_t)a->centroids) & 15) == 0) {
        // one mid-sized instance: one cooperative launch takes it from raw features to labels
        TimeScope ts__(ctx, KB_T_FIT);
        return kb_launch_fit_coop(ctx, a->N, a->D, a->K, a->iters, nullptr, a->x, a->z, a->init_rows, a->centroids, a->labels,
                                  a->dist2, a->inertia, a->rep, a->counts);
    }
    kb_status s = kb_normalize(ctx, a->B, a->N, a->D, a->x, a->z, nullptr, nullptr);
    if (s != KB_OK) return s;
    s = kb_init_centroids(ctx, a->B, a->N, a->D, a->K, a->z, a->init_rows, a->centroids);
    if (s != KB_OK) return s;
    return kb_cluster_fit(ctx, a->B, a->N, a->D, a->K, a->iters, a->z, a->centroids, a->labels, a->dist2, a->inertia,
                          a->rep, a->counts);
}

// prune, score and select: two calls, or one launch for small instances
static kb_status step_tail(kb_ctx* ctx, const kb_step_args* a, bool bound_done = false);

kb_status kb_bandit_step(kb_ctx* ctx, const kb_step_args* a) {
    if (!ctx || !a) return KB_ERR_INVALID_ARG;
    KB_COMMON(ctx, a->B, a->N);
    kb_status s = step_cluster(ctx, a);
    if (s != KB_OK) return s;
    return step_tail(ctx, a);
}

kb_status kb_bandit_step_tail(kb_ctx* ctx, const kb_step_args* a) {
    if (!ctx || !a) return KB_ERR_INVALID_ARG;
    KB_COMMON(ctx, a->B, a->N);
    return step_tail(ctx, a);
}

// bound_done: a->bound already holds the gain bound (it does not depend on the clustering): only the keep bits are due
static kb_status step_tail(kb_ctx* ctx, const kb_step_args* a, bool bound_done) {
    if (kb_step_tail_small_eligible(ctx, a)) {
        // at most 1024 candidates per instance: one CTA prunes, scores and selects for its instance
        TimeScope ts__(ctx, KB_T_SCORE);
        return kb_launch_step_tail_small(ctx, a, bound_done);
    }
    if (a->n_active || a->run_mask)
        return kb_fail(ctx, KB_ERR_UNSUPPORTED, "n_active / run_mask need a tail that runs as one CTA per instance: at most "
                                                 "1024 rows, S in {4, 8, 16, 32}, K*S <= 8192, aligned per-arm arrays");
    if (kb_step_tail_fused_eligible(ctx, a)) {
        // larger instances: the pruning rides on the statistics pass (three launches, labels and keep touched once)
        TimeScope ts__(ctx, KB_T_SCORE);
        return kb_launch_step_tail_fused(ctx, a, bound_done);
    }
    kb_status s = kb_prune(ctx, a->B, a->N, a->S, a->K, a->R, a->flops, a->bytes, a->peak_flops, a->peak_bw, a->t_incumbent,
                 a->t_cur, a->labels, a->hsig, a->target, a->theta_sat, a->keep, a->kept_count,
                 bound_done ? nullptr : a->bound);
    if (s != KB_OK) return s;
    return kb_score_select(ctx, a->B, a->N, a->K, a->S, a->score, a->labels, a->dist2, a->pulls, a->reward_sum,
                           a->keep, a->bound, a->t, a->cl_pulls, a->cl_mean, a->cl_index, a->arm_index, a->best_arm,
                           a->best_val, a->best_cluster_arm);
}

}  // extern "C"

// ---- host-buffer step ----------------------------------------------------------
namespace {
struct Carver {
    char* base;
    size_t off;
    template <typename T> T* take(size_t n) {
        T* p = reinterpret_cast<T*>(base + off);
        off += kb_align256(n * sizeof(T));
        return p;
    }
};

// device staging area of the host step; `base` may be null to only measure
size_t carve_step(char* base, const kb_step_args& h, kb_step_args* d) {
    Carver c{base, 0};
    const size_t B = h.B, N = h.N, D = h.D, K = h.K, S = h.S, R = h.R;
    kb_step_args t = h;
    float* x = c.take<float>(B * N * D);
    t.x = x; t.z = x;  // normalised in place
    t.init_rows = c.take<int32_t>(B * K);
    t.flops = c.take<float>(B * N);
    t.bytes = c.take<float>(B * N);
    t.peak_flops = c.take<float>(S);
    t.peak_bw = c.take<float>(S);
    t.t_incumbent = c.take<float>(B);
    t.t_cur = c.take<float>(B * N);
    t.hsig = c.take<float>(B * K * R);
    t.target = c.take<int32_t>(S);
    t.pulls = c.take<int32_t>(B * N * S);
    t.reward_sum = c.take<float>(B * N * S);
    t.t = c.take<int32_t>(B);
    t.centroids = c.take<float>(B * K * D);
    t.counts = c.take<int32_t>(B * K);
    t.labels = c.take<int32_t>(B * N);
    t.dist2 = c.take<float>(B * N);
    t.inertia = c.take<float>(B);
    t.rep = c.take<int32_t>(B * K);
    t.keep = c.take<uint32_t>(B * N);
    t.kept_count = c.take<uint32_t>(B);
    t.bound = h.bound ? c.take<float>(B * N * S) : nullptr;
    t.cl_pulls = c.take<float>(B * K * S);
    t.cl_mean = c.take<float>(B * K * S);
    t.cl_index = c.take<float>(B * K * S);
    t.arm_index = h.arm_index ? c.take<float>(B * N * S) : nullptr;
    t.best_arm = c.take<int32_t>(B);
    t.best_val = c.take<float>(B);
    t.best_cluster_arm = c.take<int32_t>(B);
    if (d) *d = t;
    return c.off;
}
}  // namespace

extern "C" {

kb_status kb_step_workspace_bytes(int B, int N, int D, int K, int S, int R, size_t* out) {
    if (!out || B < 0 || N < 0 || D < 0 || K < 0 || S < 0 || R < 0) return KB_ERR_INVALID_ARG;
    kb_step_args h;
    memset(&h, 0, sizeof(h));
    h.B = B; h.N = N; h.D = D; h.K = K; h.S = S; h.R = R;
    // measured with both optional outputs present
    h.bound = reinterpret_cast<float*>(1);
    h.arm_index = reinterpret_cast<float*>(1);
    size_t scratch = 0;
    kb_workspace_bytes(B, N, D, K, S, &scratch);
    *out = kb_align256(scratch) + carve_step(nullptr, h, nullptr);
    return KB_OK;
}

kb_status kb_bandit_step_host(kb_ctx* ctx, const kb_step_args* h) {
    if (!ctx || !h) return KB_ERR_INVALID_ARG;
    KB_COMMON(ctx, h->B, h->N);
    KB_REQUIRE(ctx, h->D >= 1 && h->K >= 1 && h->S >= 1 && h->R >= 1, "kb_bandit_step_host: sizes must be >= 1");
    if (h->n_active || h->run_mask)
        return kb_fail(ctx, KB_ERR_UNSUPPORTED, "kb_bandit_step_host: an expanding frontier lives on the device (n_active, "
                                                 "run_mask are for kb_bandit_step)");
    size_t scratch = 0;
    kb_workspace_bytes(h->B, h->N, h->D, h->K, h->S, &scratch);
    scratch = kb_align256(scratch);
    kb_step_args d;
    const size_t stage = carve_step(nullptr, *h, nullptr);
    if (ctx->ws_bytes < scratch + stage)
        return kb_fail(ctx, KB_ERR_WORKSPACE, "kb_bandit_step_host needs %zu bytes of workspace", scratch + stage);
    carve_step(ctx->ws + scratch, *h, &d);
    const size_t B = h->B, N = h->N, D = h->D, K = h->K, S = h->S, R = h->R;
    cudaStream_t st = ctx->stream, cs = ctx->copy_stream;
#define KB_H2D(field, count, type, stream)                                                             \
    do {                                                                                               \
        if ((count) > 0) {                                                                             \
            KB_REQUIRE(ctx, h->field, "kb_bandit_step_host: input " #field " is required");            \
            KB_CUDA(ctx, cudaMemcpyAsync(const_cast<type*>(d.field), h->field, (count) * sizeof(type), \
                                         cudaMemcpyHostToDevice, stream));                             \
        }                                                                                              \
    } while (0)
    // What normalise and the clustering read goes first, on the caller's stream.  Everything that only the
    // pruning and the scoring read (two thirds of the input bytes when S is large) is copied on a second
    // stream while the clustering runs; that stream starts behind whatever the caller's stream held before
    // this call (the staging area may still be in use by it).
    KB_CUDA(ctx, cudaEventRecord(ctx->ev_step_begin, st));
    KB_CUDA(ctx, cudaStreamWaitEvent(cs, ctx->ev_step_begin, 0));
    KB_H2D(x, B * N * D, float, st);
    KB_H2D(init_rows, B * K, int32_t, st);
    KB_H2D(flops, B * N, float, cs);
    KB_H2D(bytes, B * N, float, cs);
    KB_H2D(peak_flops, S, float, cs);
    KB_H2D(peak_bw, S, float, cs);
    KB_H2D(t_incumbent, B, float, cs);
    KB_H2D(t_cur, B * N, float, cs);
    // The gain bound B(k,s) depends on none of the clustering: once the six arrays above are up it is computed on a
    // third stream and sent back while the clustering runs (large S: a quarter of the bytes that travel).  Below a
    // megabyte the copy is shorter than what the extra launch and the two events cost the host.
    const bool early_bound = d.bound && h->bound && B * N * S * sizeof(float) >= ((size_t)1 << 20);
    if (early_bound) {
        cudaStream_t es = ctx->early_stream;
        KB_CUDA(ctx, cudaEventRecord(ctx->ev_prune_inputs, cs));
        KB_CUDA(ctx, cudaStreamWaitEvent(es, ctx->ev_prune_inputs, 0));
        ctx->stream = es;
        const kb_status sp = kb_launch_prune(ctx, d.B, d.N, d.S, d.K, d.R, d.flops, d.bytes, d.peak_flops, d.peak_bw,
                                             d.t_incumbent, d.t_cur, nullptr, nullptr, nullptr, d.theta_sat, d.keep, nullptr,
                                             d.bound);
        ctx->stream = st;
        if (sp != KB_OK) { cudaStreamSynchronize(cs); cudaStreamSynchronize(es); return sp; }
        KB_CUDA(ctx, cudaMemcpyAsync(h->bound, d.bound, B * N * S * sizeof(float), cudaMemcpyDeviceToHost, es));
        KB_CUDA(ctx, cudaEventRecord(ctx->ev_bound_done, es));
    }
    KB_H2D(hsig, B * K * R, float, cs);
    KB_H2D(target, S, int32_t, cs);
    KB_H2D(pulls, B * N * S, int32_t, cs);
    KB_H2D(reward_sum, B * N * S, float, cs);
    KB_H2D(t, B, int32_t, cs);
#undef KB_H2D
    KB_CUDA(ctx, cudaEventRecord(ctx->ev_late_inputs, cs));
    // run on the workspace's scratch part only
    char* ws_saved = ctx->ws;
    size_t bytes_saved = ctx->ws_bytes;
    ctx->ws_bytes = scratch;
    kb_status s = step_cluster(ctx, &d);
    if (s == KB_OK && cudaStreamWaitEvent(st, ctx->ev_late_inputs, 0) != cudaSuccess)
        s = kb_fail(ctx, KB_ERR_CUDA, "kb_bandit_step_host: cudaStreamWaitEvent failed");
    // (the early pass also wrote roofline-only keep bits: the real ones must come after it)
    if (s == KB_OK && early_bound && cudaStreamWaitEvent(st, ctx->ev_bound_done, 0) != cudaSuccess)
        s = kb_fail(ctx, KB_ERR_CUDA, "kb_bandit_step_host: cudaStreamWaitEvent failed");
    if (s == KB_OK) s = step_tail(ctx, &d, early_bound);
    ctx->ws = ws_saved;
    ctx->ws_bytes = bytes_saved;
    if (s != KB_OK) {
        cudaStreamSynchronize(cs);             // nothing of this call may still be writing the staging area
        cudaStreamSynchronize(ctx->early_stream);
        return s;
    }
#define KB_D2H(field, count, type)                                                                          \
    do {                                                                                                    \
        if (h->field && (count) > 0)                                                                        \
            KB_CUDA(ctx, cudaMemcpyAsync(h->field, d.field, (count) * sizeof(type), cudaMemcpyDeviceToHost, st)); \
    } while (0)
    KB_D2H(z, B * N * D, float);
    KB_D2H(centroids, B * K * D, float);
    KB_D2H(counts, B * K, int32_t);
    KB_D2H(labels, B * N, int32_t);
    KB_D2H(dist2, B * N, float);
    KB_D2H(inertia, B, float);
    KB_D2H(rep, B * K, int32_t);
    KB_D2H(keep, B * N, uint32_t);
    KB_D2H(kept_count, B, uint32_t);
    if (!early_bound) KB_D2H(bound, B * N * S, float);
    KB_D2H(cl_pulls, B * K * S, float);
    KB_D2H(cl_mean, B * K * S, float);
    KB_D2H(cl_index, B * K * S, float);
    KB_D2H(arm_index, B * N * S, float);
    KB_D2H(best_arm, B, int32_t);
    KB_D2H(best_val, B, float);
    KB_D2H(best_cluster_arm, B, int32_t);
#undef KB_D2H
    // this call synchronises anyway: the status word comes back with the results
    int word = 0;
    KB_CUDA(ctx, cudaMemcpyAsync(&word, ctx->dev_status, sizeof(int), cudaMemcpyDeviceToHost, st));
    KB_CUDA(ctx, cudaStreamSynchronize(st));
    return kb_status_from_device_word(ctx, word, true);
}

}  // extern "C"
