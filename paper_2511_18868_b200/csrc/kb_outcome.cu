// kb_record_outcome: the outcome of one iteration (Sec. 2.2 "Formal Model": r_t = Clip((L(k_t) -
// L(k'_t)) / L(k_t), 0, 1); Algorithm 1, "Generation & update": N <- N + 1, mu <- mu + (r_t - mu) / N
// for the chosen pair).
//
// The statistics live per arm as (pulls, reward_sum); kb_score_select forms N_{i,s} and mu_{i,s}
// per cluster from them in closed form, so a re-clustering re-aggregates the history.  The update
// of the pair (I_t, S_t) through its drawn member k_t is pulls[k_t][S_t] += 1,
// reward_sum[k_t][S_t] += r_t: one thread per instance, three words touched.  The kernel exists so
// that selection, draw and update of B lock-step searches stay on the device, in one stream or one
// CUDA graph, with no host round trip between them.
#include "kb_internal.cuh"

namespace {

__global__ void record_outcome_kernel(int B, int N, int S, int failures_count, const int32_t* __restrict__ member,
                                      const int32_t* __restrict__ cluster_arm, const float* __restrict__ t_cur,
                                      const float* __restrict__ t_new, const int32_t* __restrict__ verified,
                                      int32_t* __restrict__ pulls, float* __restrict__ reward_sum,
                                      int32_t* __restrict__ t, float* __restrict__ reward,
                                      int* __restrict__ dev_status) {
    kb_grid_dependency_wait();
    const int b = blockIdx.x * blockDim.x + threadIdx.x;
    if (b >= B) return;
    t[b] += 1;                                   // the loop index of Algorithm 1 advances in every case
    float r = 0.f;
    const int k = member[b];
    const int ca = cluster_arm[b];
    if (k >= 0) {
        if (k >= N || ca < 0) {
            atomicOr(dev_status, 4);
        } else {
            const bool ok = verified ? verified[b] != 0 : true;
            if (ok || failures_count) {
                if (ok) {
                    const float L = t_cur[(size_t)b * N + k], Ln = t_new[b];
                    r = L > 0.f ? (L - Ln) / L : 0.f;
                    r = r > 0.f ? r : 0.f;       // regressions and NaN
                    r = r < 1.f ? r : 1.f;
                }
                const size_t i = ((size_t)b * N + k) * S + (ca % S);
                pulls[i] += 1;
                reward_sum[i] += r;
            }
        }
    }
    if (reward) reward[b] = r;
}

}  // namespace

kb_status kb_launch_record_outcome(kb_ctx* ctx, int B, int N, int S, int failures_count, const int32_t* member,
                                   const int32_t* cluster_arm, const float* t_cur, const float* t_new,
                                   const int32_t* verified, int32_t* pulls, float* reward_sum, int32_t* t,
                                   float* reward) {
    if (B == 0) return KB_OK;
    kb_launch(record_outcome_kernel, (B + 127) / 128, 128, 0, ctx->stream, B, N, S, failures_count, member, cluster_arm,
              t_cur, t_new, verified, pulls, reward_sum, t, reward, ctx->dev_status);
    KB_LAUNCH_CHECK(ctx, "record_outcome_kernel");
    return KB_OK;
}
