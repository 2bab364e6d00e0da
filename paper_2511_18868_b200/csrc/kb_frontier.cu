// The expanding frontier (Sec. 2.2: the action space grows with the frontier; Algorithm 1: "P <- P U {k'_t}"
// inside "if Verify(k'_t)", and the test "t mod tau = 0 and |P| >= 2K"): three small kernels that keep the
// frontier's growth, the re-cluster decision and the clusters' signatures on the device, so that a search loop
// never has to bring the frontier back to the host.
#include "kb_internal.cuh"

namespace {

struct AppendArgs {
    int N_cap, D, S, R;
    const int32_t *verified, *parent;
    const float *x_new, *t_new, *flops_new, *bytes_new, *h_new;
    int32_t* n_active;
    float *x, *t_cur, *flops, *bytes, *h_cand;
    int32_t* labels;
    float* dist2;
    int32_t* pulls;
    float *reward_sum, *t_inc;
    int32_t* appended;
    int* dev_status;
};

// one warp per search: lane 0 decides, all lanes copy the row
__global__ void __launch_bounds__(32) append_candidate_kernel(const AppendArgs a) {
    kb_grid_dependency_wait();
    const int b = blockIdx.x, lane = threadIdx.x;
    const int p = a.parent[b];
    const int n = a.n_active[b];
    int row = -1;
    if (p >= 0 && (!a.verified || a.verified[b] != 0)) {
        if (n < 0 || n > a.N_cap || p >= n) {
            if (lane == 0) atomicOr(a.dev_status, KB_STATUS_BAD_INDEX);
        } else if (n == a.N_cap) {
            if (lane == 0) atomicOr(a.dev_status, KB_STATUS_FRONTIER_FULL);
        } else {
            row = n;
        }
    }
    if (lane == 0 && a.appended) a.appended[b] = row;
    if (row < 0) return;
    const size_t i = (size_t)b * a.N_cap + row, ip = (size_t)b * a.N_cap + p;
    for (int d = lane; d < a.D; d += 32) a.x[i * a.D + d] = a.x_new[(size_t)b * a.D + d];
    for (int s = lane; s < a.S; s += 32) { a.pulls[i * a.S + s] = 0; a.reward_sum[i * a.S + s] = 0.f; }
    if (a.h_cand && a.h_new)
        for (int r = lane; r < a.R; r += 32) a.h_cand[i * a.R + r] = a.h_new[(size_t)b * a.R + r];
    if (lane == 0) {
        const float tn = a.t_new[b];
        a.t_cur[i] = tn;
        if (a.flops && a.flops_new) a.flops[i] = a.flops_new[b];
        if (a.bytes && a.bytes_new) a.bytes[i] = a.bytes_new[b];
        a.labels[i] = a.labels[ip];
        if (a.dist2) a.dist2[i] = a.dist2[ip];
        if (a.t_inc && tn < a.t_inc[b]) a.t_inc[b] = tn;
        a.n_active[b] = n + 1;
    }
}

__global__ void __launch_bounds__(256) recluster_due_kernel(int B, int tau, int K, const int32_t* __restrict__ t,
                                                            const int32_t* __restrict__ n_active,
                                                            int32_t* __restrict__ due, int32_t* __restrict__ any_due) {
    kb_grid_dependency_wait();
    __shared__ int s_any;
    if (threadIdx.x == 0) s_any = 0;
    __syncthreads();
    int mine = 0;
    for (int b = threadIdx.x; b < B; b += blockDim.x) {
        const int d = (t[b] % tau == 0 && n_active[b] >= 2 * K) ? 1 : 0;
        due[b] = d;
        mine |= d;
    }
    if (mine) atomicOr(&s_any, 1);
    __syncthreads();
    if (threadIdx.x == 0 && any_due) *any_due = s_any;
}

__global__ void __launch_bounds__(128) signatures_from_reps_kernel(int N, int K, int R, const int32_t* __restrict__ rep,
                                                                   const float* __restrict__ h_cand,
                                                                   const int32_t* __restrict__ run_mask,
                                                                   float* __restrict__ hsig, int* __restrict__ dev_status) {
    kb_grid_dependency_wait();
    const int b = blockIdx.y;
    if (run_mask && run_mask[b] == 0) return;
    const int e = blockIdx.x * blockDim.x + threadIdx.x;
    if (e >= K * R) return;
    const int i = e / R, r = e - i * R;
    const int k = rep[(size_t)b * K + i];
    float v = INFINITY;                                              // an empty cluster is saturated on every resource
    if (k >= N) atomicOr(dev_status, KB_STATUS_BAD_INDEX);
    else if (k >= 0) v = h_cand[((size_t)b * N + k) * R + r];
    hsig[(size_t)b * K * R + e] = v;
}

}  // namespace

kb_status kb_launch_append_candidate(kb_ctx* ctx, int B, int N_cap, int D, int S, int R, const int32_t* verified,
                                     const int32_t* parent, const float* x_new, const float* t_new, const float* flops_new,
                                     const float* bytes_new, const float* h_new, int32_t* n_active, float* x, float* t_cur,
                                     float* flops, float* bytes, float* h_cand, int32_t* labels, float* dist2,
                                     int32_t* pulls, float* reward_sum, float* t_inc, int32_t* appended) {
    if (B == 0) return KB_OK;
    AppendArgs a;
    a.N_cap = N_cap; a.D = D; a.S = S; a.R = R;
    a.verified = verified; a.parent = parent; a.x_new = x_new; a.t_new = t_new; a.flops_new = flops_new;
    a.bytes_new = bytes_new; a.h_new = h_new; a.n_active = n_active; a.x = x; a.t_cur = t_cur; a.flops = flops;
    a.bytes = bytes; a.h_cand = h_cand; a.labels = labels; a.dist2 = dist2; a.pulls = pulls; a.reward_sum = reward_sum;
    a.t_inc = t_inc; a.appended = appended; a.dev_status = ctx->dev_status;
    kb_launch(append_candidate_kernel, B, 32, 0, ctx->stream, a);
    KB_LAUNCH_CHECK(ctx, "append_candidate_kernel");
    return KB_OK;
}

kb_status kb_launch_recluster_due(kb_ctx* ctx, int B, int tau, int K, const int32_t* t, const int32_t* n_active,
                                  int32_t* due, int32_t* any_due) {
    kb_launch(recluster_due_kernel, 1, 256, 0, ctx->stream, B, tau, K, t, n_active, due, any_due);
    KB_LAUNCH_CHECK(ctx, "recluster_due_kernel");
    return KB_OK;
}

kb_status kb_launch_signatures_from_reps(kb_ctx* ctx, int B, int N, int K, int R, const int32_t* rep, const float* h_cand,
                                         const int32_t* run_mask, float* hsig) {
    if (B == 0) return KB_OK;
    kb_launch(signatures_from_reps_kernel, dim3((K * R + 127) / 128, B), 128, 0, ctx->stream, N, K, R, rep, h_cand, run_mask,
              hsig, ctx->dev_status);
    KB_LAUNCH_CHECK(ctx, "signatures_from_reps_kernel");
    return KB_OK;
}
