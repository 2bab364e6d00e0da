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
//
// Given the K x S cluster tables (cl_pulls, cl_mean) the same thread also applies Algorithm 1's own two lines
// to the chosen pair, so the tables stay current and the next pair can be chosen by kb_select_pair (below) from
// K*S entries, without a pass over the arms.
#include "kb_internal.cuh"

namespace {

__global__ void record_outcome_kernel(int B, int N, int K, int S, int failures_count, const int32_t* __restrict__ member,
                                      const int32_t* __restrict__ cluster_arm, const float* __restrict__ t_cur,
                                      const float* __restrict__ t_new, const int32_t* __restrict__ verified,
                                      int32_t* __restrict__ pulls, float* __restrict__ reward_sum,
                                      int32_t* __restrict__ t, float* __restrict__ reward,
                                      float* __restrict__ cl_pulls, float* __restrict__ cl_mean,
                                      int* __restrict__ dev_status) {
    kb_grid_dependency_wait();
    const int b = blockIdx.x * blockDim.x + threadIdx.x;
    if (b >= B) return;
    t[b] += 1;                                   // the loop index of Algorithm 1 advances in every case
    float r = 0.f;
    const int k = member[b];
    const int ca = cluster_arm[b];
    if (k >= 0) {
        if (k >= N || ca < 0 || (cl_pulls && ca >= K * S)) {
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
                if (cl_pulls) {
                    // the cluster tables kept alongside: Algorithm 1's two lines, literally
                    const size_t p = (size_t)b * K * S + ca;
                    const float n = cl_pulls[p] + 1.f;
                    const float mu = cl_mean[p];
                    cl_pulls[p] = n;
                    cl_mean[p] = mu + (r - mu) / n;
                }
            }
        }
    }
    if (reward) reward[b] = r;
}

}  // namespace

kb_status kb_launch_record_outcome(kb_ctx* ctx, int B, int N, int K, int S, int failures_count, const int32_t* member,
                                   const int32_t* cluster_arm, const float* t_cur, const float* t_new,
                                   const int32_t* verified, int32_t* pulls, float* reward_sum, int32_t* t,
                                   float* reward, float* cl_pulls, float* cl_mean) {
    if (B == 0) return KB_OK;
    kb_launch(record_outcome_kernel, (B + 127) / 128, 128, 0, ctx->stream, B, N, K, S, failures_count, member, cluster_arm,
              t_cur, t_new, verified, pulls, reward_sum, t, reward, cl_pulls, cl_mean, ctx->dev_status);
    KB_LAUNCH_CHECK(ctx, "record_outcome_kernel");
    return KB_OK;
}

// ---- the masked-UCB choice of the pair from the cluster tables (Sec. 3.4; Algorithm 1, "Select (I_t, S_t)") ----
namespace {
constexpr int SP_MAX_T = 1024;   // one CTA per instance; its width follows K*S (a thread should see few entries:
                                 // each costs a dependent round trip to L2 for its table entries and its mask)
__global__ void __launch_bounds__(SP_MAX_T)
select_pair_kernel(int K, int S, int R, float c, const float* __restrict__ cl_pulls, const float* __restrict__ cl_mean,
                   const int32_t* __restrict__ t, const float* __restrict__ hsig, const int32_t* __restrict__ target,
                   float theta, float* __restrict__ cl_index, int32_t* __restrict__ pair, int* __restrict__ dev_status) {
    kb_grid_dependency_wait();
    __shared__ unsigned long long s_red[SP_MAX_T / 32];
    const int b = blockIdx.x, tid = threadIdx.x, KS = K * S, T = blockDim.x;
    const float lnt = logf((float)t[b]);
    unsigned long long best = 0ull;
    for (int e = tid; e < KS; e += T) {
        const size_t o = (size_t)b * KS + e;
        const float u = cl_mean[o] + c * sqrtf(lnt / cl_pulls[o]);
        if (cl_index) cl_index[o] = u;
        bool valid = true;
        if (hsig) {
            const int i = e / S, col = target[e - i * S];
            if (col < 0 || col >= R) { atomicOr(dev_status, 2); valid = false; }
            else valid = hsig[((size_t)b * K + i) * R + col] < theta;
        }
        if (valid) {
            const unsigned long long key = ((unsigned long long)kb_orderable(u) << 32) | (0xffffffffu - (unsigned)e);
            best = key > best ? key : best;
        }
    }
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) {
        const unsigned long long other = __shfl_xor_sync(0xffffffffu, best, o);
        best = other > best ? other : best;
    }
    if ((tid & 31) == 0) s_red[tid >> 5] = best;
    __syncthreads();
    if (tid == 0) {
        for (int w = 1; w < T / 32; ++w) best = s_red[w] > best ? s_red[w] : best;
        pair[b] = best ? (int32_t)(0xffffffffu - (unsigned)(best & 0xffffffffull)) : -1;
    }
}
}  // namespace

kb_status kb_launch_select_pair(kb_ctx* ctx, int B, int K, int S, int R, float c, const float* cl_pulls,
                                const float* cl_mean, const int32_t* t, const float* hsig, const int32_t* target,
                                float theta_sat, float* cl_index, int32_t* pair) {
    if (B == 0) return KB_OK;
    long ks = (long)K * S;
    int threads = (int)(ks >= SP_MAX_T ? SP_MAX_T : ((ks + 31) / 32) * 32);
    if (threads < 32) threads = 32;
    kb_launch(select_pair_kernel, B, threads, 0, ctx->stream, K, S, R, c, cl_pulls, cl_mean, t, hsig, target, theta_sat, cl_index,
              pair, ctx->dev_status);
    KB_LAUNCH_CHECK(ctx, "select_pair_kernel");
    return KB_OK;
}
