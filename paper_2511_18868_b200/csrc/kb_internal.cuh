// Internal declarations shared by the CUDA translation units of libkb.
#pragma once

#include <cuda_runtime.h>
#include <stdint.h>
#include <stdio.h>

#include "kb.h"

struct kb_ctx {
    int device;
    cudaStream_t stream;
    int sm_count;
    int max_smem_optin;   // bytes of dynamic shared memory a block may opt into
    int coop_launch;      // the device supports cooperative launches
    char* ws;             // caller's workspace (device)
    size_t ws_bytes;
    int* dev_status;      // device status word (owned)
    cudaStream_t copy_stream;       // host-buffer step: copies of the late inputs (owned)
    cudaStream_t early_stream;      // host-buffer step: the gain bound, computed and sent back while the clustering runs (owned)
    cudaEvent_t ev_step_begin, ev_late_inputs, ev_prune_inputs, ev_bound_done;
    uint64_t launches;    // kernels queued so far
    uint64_t memsets;     // memset nodes queued so far
    // optional per-call event timing
    bool timing;
    cudaEvent_t* ev;      // 2 * KB_EV_PAIRS events
    int ev_used;          // pairs in use
    unsigned char* ev_class;
    // assign path control: 0 = automatic, 1 = row-wise FFMA, 2 = tensor cores
    int assign_path;
    int last_assign_path;  // path the most recent kb_cluster_assign took (1 or 2; 0 = nothing ran)
    int last_assign_presplit;   // 1: that assignment multiplied out of the pre-split image of Z
    float tc_eps;          // near-tie bound of the tensor path, relative to ||z||^2 + ||c||^2
    // pre-split fp16 image of a matrix Z that a running fit keeps in the workspace (zs_src == nullptr: none)
    const float* zs_src;
    int zs_B, zs_N, zs_D;
    const unsigned char* zs_img;
    const float* zs_info;
    // accumulators (sums, then counts) that a running tensor-path fit sets aside for its updates, behind the
    // scratch of the calls: the assignment's fix-up kernel clears them, so the update needs no clearing launch
    char* fit_acc;               // null outside such a fit
    size_t fit_acc_bytes;
    int fit_acc_clean;           // 1: cleared since the last update used them
    // test hooks of the bounded device-side waits (kb_debug_wait_limit): 0 / 0 in normal operation
    unsigned dbg_wait_limit;     // polls after which a wait gives up (0: the kernels' own limits)
    int dbg_skip_arrival;        // 1: one participant never arrives, so the others' waits run out
    char err[256];
};
#define KB_EV_PAIRS 4096

// ---- error plumbing ---------------------------------------------------------
kb_status kb_fail(kb_ctx* ctx, kb_status s, const char* fmt, ...);
kb_status kb_status_from_device_word(kb_ctx* ctx, int word, bool contract_bits_too);

#define KB_CUDA(ctx, expr)                                                                     \
    do {                                                                                       \
        cudaError_t e__ = (expr);                                                              \
        if (e__ != cudaSuccess)                                                                \
            return kb_fail(ctx, KB_ERR_CUDA, "%s: %s", #expr, cudaGetErrorString(e__));        \
    } while (0)

#define KB_LAUNCH_CHECK(ctx, name)                                                             \
    do {                                                                                       \
        cudaError_t e__ = cudaGetLastError();                                                  \
        if (e__ != cudaSuccess)                                                                \
            return kb_fail(ctx, KB_ERR_CUDA, "launch of %s: %s", name, cudaGetErrorString(e__)); \
        (ctx)->launches++;                                                                     \
    } while (0)

#define KB_MEMSET(ctx, ptr, val, bytes)                                                        \
    do {                                                                                       \
        KB_CUDA(ctx, cudaMemsetAsync(ptr, val, bytes, (ctx)->stream));                         \
        (ctx)->memsets++;                                                                      \
    } while (0)

#define KB_REQUIRE(ctx, cond, msg)                                                             \
    do {                                                                                       \
        if (!(cond)) return kb_fail(ctx, KB_ERR_INVALID_ARG, "%s", msg);                       \
    } while (0)

// optional event pair around a single kernel (while per-call timing is on); returns the slot or -1
static inline int kb_time_begin(kb_ctx* ctx, int cls) {
    if (!ctx->timing || ctx->ev_used >= KB_EV_PAIRS) return -1;
    const int slot = ctx->ev_used++;
    ctx->ev_class[slot] = (unsigned char)cls;
    cudaEventRecord(ctx->ev[2 * slot], ctx->stream);
    return slot;
}
static inline void kb_time_end(kb_ctx* ctx, int slot) {
    if (slot >= 0) cudaEventRecord(ctx->ev[2 * slot + 1], ctx->stream);
}

// ---- workspace ------------------------------------------------------------------
// Every call carves its scratch from the start of the workspace and clears the
// control words it relies on, so nothing in the workspace has to survive from
// one call to the next.  kb_workspace_bytes is the largest of these needs.
size_t kb_ws_need_normalize(int B, int N, int D);
size_t kb_ws_need_assign(int B, int N, int D, int K);
size_t kb_ws_need_assign_tc(int B, int N, int D, int K);
size_t kb_ws_need_zsplit(int B, int N, int D, int K);
bool kb_step_tail_small_eligible(const kb_ctx* ctx, const kb_step_args* a);
bool kb_score_small_eligible(const kb_ctx* ctx, int B, int N, int K, int S, kb_score_params p, const float* dist2,
                             const int32_t* pulls, const float* reward_sum, const float* bound, const float* arm_index);
kb_status kb_launch_score_small(kb_ctx* ctx, int B, int N, int K, int S, kb_score_params p, const int32_t* labels,
                                const float* dist2, const int32_t* pulls, const float* reward_sum, const uint32_t* keep,
                                const float* bound, const int32_t* t, float* cl_pulls, float* cl_mean, float* cl_index,
                                float* arm_index, int32_t* best_arm, float* best_val, int32_t* best_cluster_arm);
kb_status kb_launch_step_tail_small(kb_ctx* ctx, const kb_step_args* a, bool bound_done = false);
bool kb_step_tail_fused_eligible(const kb_ctx* ctx, const kb_step_args* a);
kb_status kb_launch_step_tail_fused(kb_ctx* ctx, const kb_step_args* a, bool bound_done = false);
kb_status kb_zsplit_prepare(kb_ctx* ctx, char* img, int B, int N, int D, int K, const float* z);
void kb_zsplit_forget(kb_ctx* ctx);
bool kb_assign_tc_supported(const kb_ctx* ctx, int B, int D, int K);
bool kb_assign_tc_eligible(const kb_ctx* ctx, int B, int N, int D, int K);
kb_status kb_launch_assign_tc(kb_ctx* ctx, char* ws, int B, int N, int D, int K, const float* z, const float* c,
                              int32_t* labels, float* approx, int* flagged, float eps);
kb_status kb_launch_assign_finish(kb_ctx* ctx, int B, int N, int D, int K, const float* z, const float* c,
                                  const int32_t* labels, float* dist2, double* ws_inertia,
                                  unsigned long long* ws_rep);
bool kb_fit_fused_eligible(const kb_ctx* ctx, int B, int N, int D, int K);
bool kb_fit_coop_eligible(const kb_ctx* ctx, int B, int N, int D, int K);
size_t kb_ws_need_fit_coop(int B, int N, int D, int K);
kb_status kb_launch_fit_coop(kb_ctx* ctx, int N, int D, int K, int iters, const float* z, const float* xraw, float* zout,
                             const int32_t* init_rows, float* cent, int32_t* labels, float* dist2, float* inertia,
                             int32_t* rep, int32_t* counts);
kb_status kb_launch_fit_fused(kb_ctx* ctx, int B, int N, int D, int K, int iters, const float* z, const float* xraw,
                              float* zout, const int32_t* init_rows, float* cent, int32_t* labels, float* dist2,
                              float* inertia, int32_t* rep, int32_t* counts, const int32_t* n_active = nullptr,
                              const int32_t* run_mask = nullptr, float tol = -1.f, int32_t* n_iter = nullptr);
// every coordinate of the centroid of an unused cluster (rows = -1 in kb_init_centroids / init_rows): farther from any
// data than any real centroid, finite when squared and summed over a few hundred features
#define KB_UNUSED_CENTROID 1e18f
size_t kb_ws_need_update(int B, int N, int D, int K);
size_t kb_ws_need_fit_acc(int B, int D, int K);
size_t kb_ws_need_score(int B, int N, int K, int S);
#define KB_NORM_MAXG 1024
int kb_norm_blocks_per_instance(int B, int N);
static inline size_t kb_align256(size_t v) { return (v + 255) & ~(size_t)255; }

// ---- per-call launchers (each validates nothing: the API layer does) ----------
kb_status kb_launch_normalize(kb_ctx*, int B, int N, int D, const float* x, float* z, float* mean, float* scale);
kb_status kb_launch_prune(kb_ctx*, int B, int N, int S, int K, int R, const float* flops, const float* bytes,
                          const float* peak_flops, const float* peak_bw, const float* t_inc, const float* t_cur,
                          const int32_t* labels, const float* hsig, const int32_t* target, float theta,
                          uint32_t* keep, uint32_t* kept, float* bound);
kb_status kb_launch_assign(kb_ctx*, int B, int N, int D, int K, const float* z, const float* c, int32_t* labels,
                           float* dist2, float* inertia, int32_t* rep);
kb_status kb_launch_update(kb_ctx*, int B, int N, int D, int K, const float* z, const int32_t* labels,
                           float* c, int32_t* counts);
kb_status kb_launch_score(kb_ctx*, int B, int N, int K, int S, kb_score_params p, const int32_t* labels,
                          const float* dist2, const int32_t* pulls, const float* reward_sum, const uint32_t* keep,
                          const float* bound, const int32_t* t, float* cl_pulls, float* cl_mean, float* cl_index,
                          float* arm_index, int32_t* best_arm, float* best_val, int32_t* best_cluster_arm);
kb_status kb_launch_record_outcome(kb_ctx*, int B, int N, int K, int S, int failures_count, const int32_t* member,
                                   const int32_t* cluster_arm, const float* t_cur, const float* t_new,
                                   const int32_t* verified, int32_t* pulls, float* reward_sum, int32_t* t,
                                   float* reward, float* cl_pulls, float* cl_mean);
kb_status kb_launch_select_pair(kb_ctx*, int B, int K, int S, int R, float c, const float* cl_pulls, const float* cl_mean,
                                const int32_t* t, const float* hsig, const int32_t* target, float theta_sat,
                                float* cl_index, int32_t* pair);
kb_status kb_launch_cluster_radius(kb_ctx*, int B, int N, int K, const int32_t* labels, const float* dist2, float* radius);
size_t kb_ws_need_topm(int B, int M);
kb_status kb_launch_top_m(kb_ctx*, int B, int NS, int M, const float* arm_index, int32_t* top_arm, float* top_val);
kb_status kb_launch_best_restart(kb_ctx*, int G, int n_init, const float* inertia, int32_t* best);
size_t kb_ws_need_seed(int B, int N, int K);
kb_status kb_launch_seed_kmeanspp(kb_ctx*, int B, int N, int D, int K, const float* z, uint64_t seed, int32_t* rows);
size_t kb_ws_need_sample(int B);
kb_status kb_launch_sample_member(kb_ctx*, int B, int N, int K, int S, int R, const int32_t* labels,
                                  const int32_t* cluster_arm, const float* h_cand, const int32_t* target,
                                  float theta_sat, uint64_t seed, const int32_t* t, int32_t* member,
                                  float* member_val);
kb_status kb_launch_init_centroids(kb_ctx*, int B, int N, int D, int K, const float* z, const int32_t* rows,
                                   float* c);
kb_status kb_launch_append_candidate(kb_ctx* ctx, int B, int N_cap, int D, int S, int R, const int32_t* verified,
                                     const int32_t* parent, const float* x_new, const float* t_new, const float* flops_new,
                                     const float* bytes_new, const float* h_new, int32_t* n_active, float* x, float* t_cur,
                                     float* flops, float* bytes, float* h_cand, int32_t* labels, float* dist2,
                                     int32_t* pulls, float* reward_sum, float* t_inc, int32_t* appended);
kb_status kb_launch_recluster_due(kb_ctx* ctx, int B, int tau, int K, const int32_t* t, const int32_t* n_active,
                                  int32_t* due, int32_t* any_due);
kb_status kb_launch_signatures_from_reps(kb_ctx* ctx, int B, int N, int K, int R, const int32_t* rep, const float* h_cand,
                                         const int32_t* run_mask, float* hsig);

// Opts a kernel into more than 48 KB of dynamic shared memory when it needs it.
#define KB_SMEM_OPTIN(ctx, kernel, bytes)                                                        \
    do {                                                                                         \
        if ((bytes) > 48 * 1024)                                                                 \
            KB_CUDA(ctx, cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)(bytes))); \
    } while (0)

// ---- launches with programmatic dependent launch ------------------------------
// Every kernel of the library is launched with the programmatic-stream-serialization attribute and
// begins with kb_grid_dependency_wait(): the next kernel's blocks may be scheduled, and run their
// prologue up to that wait, while the previous kernel drains, which hides most of the launch gap
// between the many short dependent kernels of a Lloyd iteration.  The wait returns when the
// preceding kernel has completed and its writes are visible; as every kernel takes it before
// touching global memory, completion is transitive along the stream.
#ifdef __CUDACC__
__device__ __forceinline__ void kb_grid_dependency_wait() { asm volatile("griddepcontrol.wait;" ::: "memory"); }

template <typename... KArgs, typename... Args>
inline cudaError_t kb_launch(void (*kernel)(KArgs...), dim3 grid, dim3 block, size_t smem, cudaStream_t stream,
                             Args&&... args) {
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = grid;
    cfg.blockDim = block;
    cfg.dynamicSmemBytes = smem;
    cfg.stream = stream;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr;
    cfg.numAttrs = 1;
    return cudaLaunchKernelEx(&cfg, kernel, KArgs(args)...);
}
#endif

// ---- small device helpers -----------------------------------------------------
#ifdef __CUDACC__
__device__ __forceinline__ float kb_warp_sum(float v) {
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
    return v;
}
__device__ __forceinline__ double kb_warp_sum(double v) {
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
    return v;
}
// a / d with r = 1/d (correctly rounded): one residual step on the first estimate
__device__ __forceinline__ float kb_div_by(float a, float d, float r) {
    const float q0 = a * r;
    const float e = fmaf(-q0, d, a);
    return fmaf(e, r, q0);     // d = 0 or a non-finite operand gives NaN here, which the callers map like 0/0
}
// Philox4x32 with 10 rounds (Salmon et al., SC'11): first output word only.
__device__ __forceinline__ uint32_t kb_philox4x32_10_word0(uint32_t c0, uint32_t c1, uint32_t c2, uint32_t c3,
                                                       uint32_t k0, uint32_t k1) {
    constexpr uint32_t M0 = 0xD2511F53u, M1 = 0xCD9E8D57u, W0 = 0x9E3779B9u, W1 = 0xBB67AE85u;
#pragma unroll
    for (int r = 0; r < 10; ++r) {
        const uint32_t hi0 = __umulhi(M0, c0), lo0 = M0 * c0;
        const uint32_t hi1 = __umulhi(M1, c2), lo1 = M1 * c2;
        c0 = hi1 ^ c1 ^ k0;
        c1 = lo1;
        c2 = hi0 ^ c3 ^ k1;
        c3 = lo0;
        k0 += W0;
        k1 += W1;
    }
    return c0;
}
// the uniform in (0, 1) the draws use: 23 bits of the word, centred, exact in fp32
__device__ __forceinline__ float kb_uniform23(uint32_t w) { return ((float)(w >> 9) + 0.5f) * (1.0f / 8388608.0f); }
// monotone map float -> uint32 (larger float <=> larger uint)
__device__ __forceinline__ uint32_t kb_orderable(float f) {
    uint32_t u = __float_as_uint(f);
    return (u & 0x80000000u) ? ~u : (u | 0x80000000u);
}
__device__ __forceinline__ float kb_from_orderable(uint32_t u) {
    return __uint_as_float((u & 0x80000000u) ? (u & 0x7fffffffu) : ~u);
}
#endif
