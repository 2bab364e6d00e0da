// kb_prune + kb_score_select for small instances inside the whole-step drivers: one CTA per
// instance, ONE launch instead of six kernels and two clears.
//
// With a few hundred candidates per instance the two calls are launch latency (a tiny step) or
// re-read what the other has just touched (many small instances).  Here a CTA walks its
// instance's arms twice:
//   pass 1  per (candidate, four strategies): the roofline floor against the incumbent and the
//           saturation mask (Sec. 3.4) give the keep bits, Assumption 1 gives the gain bound;
//           pulls and rewards are added into per-(cluster, strategy) tables in shared memory --
//           the arithmetic of prune_vec_kernel and score_stats_kernel, in the same order per arm;
//   table   N, mu and U_cl per (cluster, strategy) from the shared tables (masked-UCB equation),
//           the cluster-level argmax;
//   pass 2  the per-arm index U_cl + L sqrt(dist2) (Assumption 2), optional cap, mask, store,
//           the arm-level argmax -- the arithmetic of score_arms_kernel.
// Both argmax results are packed keys (value, then lowest index) reduced inside the CTA.
#include "kb_internal.cuh"

namespace {

constexpr int ST_T = 256;

struct TailArgs {
    int N, S, K, R;
    int write_bound;        // 0: bound is there already (it does not depend on the clustering) and is only read
    float theta;
    kb_score_params prm;
    const float *flops, *bytes, *peak_flops, *peak_bw, *t_inc, *t_cur, *hsig, *dist2, *reward_sum;
    const int32_t *labels, *target, *pulls, *t;
    uint32_t *keep, *kept;
    float *bound, *cl_pulls, *cl_mean, *cl_index, *arm_index, *best_val;
    int32_t *best_arm, *best_cluster_arm;
    const int32_t *n_active, *run_mask;   // expanding frontier: candidates per instance (of N rows), instances to run
    int* dev_status;
};

__device__ __forceinline__ unsigned long long block_max_key(unsigned long long v, unsigned long long* s_red) {
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) {
        const unsigned long long other = __shfl_xor_sync(0xffffffffu, v, o);
        v = other > v ? other : v;
    }
    __syncthreads();                                     // s_red may still be read from an earlier reduction
    if ((threadIdx.x & 31) == 0) s_red[threadIdx.x >> 5] = v;
    __syncthreads();
    v = s_red[0];
#pragma unroll
    for (int w = 1; w < ST_T / 32; ++w) v = s_red[w] > v ? s_red[w] : v;
    return v;
}

// PRUNE = false: the keep bits are an input (a.keep, null = every arm valid) and nothing of the pruning is computed
// or written: the same kernel then is kb_score_select for small instances.
template <bool PRUNE>
__global__ void __launch_bounds__(ST_T)
step_tail_small_kernel(const TailArgs a) {
    kb_grid_dependency_wait();
    extern __shared__ __align__(16) unsigned char sraw[];
    // An expanding frontier: the arrays have a.N rows per instance of which the first n_active[b] are candidates
    // (N below; NP is the pitch); an instance whose run_mask entry is 0 is left exactly as it is.
    if (a.run_mask && a.run_mask[blockIdx.x] == 0) return;
    const int NP = a.N, S = a.S, K = a.K, KS = K * S;
    const int N = a.n_active ? min(max(a.n_active[blockIdx.x], 0), NP) : NP;
    int* sp = reinterpret_cast<int*>(sraw);                      // [K][S] pull sums
    float* sr = reinterpret_cast<float*>(sraw) + KS;             // [K][S] reward sums
    float* tab = sr + KS;                                        // [K][S] U_cl
    unsigned* sa = reinterpret_cast<unsigned*>(tab + KS);        // [K] any kept member arm, bit s
    unsigned* skeep = sa + K;                                    // [N] keep bits of this instance
    __shared__ float s_rP[32], s_rW[32];
    __shared__ unsigned s_cnt[ST_T / 32];
    __shared__ unsigned long long s_red[ST_T / 32];
    const int b = blockIdx.x, tid = threadIdx.x, lane = tid & 31;
    const int vps = S >> 2;                                      // lanes per candidate: 1, 2, 4 or 8
    const int q = tid % vps, rstep = ST_T / vps;
    const int trips = (N + rstep - 1) / rstep;                   // the same for every thread: shuffles stay warp-wide

    for (int e = tid; e < 2 * KS; e += ST_T) sp[e] = 0;          // int 0 == float +0 bit pattern
    for (int j = tid; j < K; j += ST_T) sa[j] = 0;
    if (PRUNE && tid < S) {
        s_rP[tid] = 1.f / a.peak_flops[tid];
        s_rW[tid] = 1.f / a.peak_bw[tid];
    }
    __syncthreads();
    float P[4], W[4], rP[4], rW[4];
    int tg[4];
    float tinc = 0.f;
    if (PRUNE) {
#pragma unroll
        for (int i = 0; i < 4; ++i) {
            P[i] = a.peak_flops[4 * q + i];
            W[i] = a.peak_bw[4 * q + i];
            rP[i] = s_rP[4 * q + i];
            rW[i] = s_rW[4 * q + i];
            int t = a.target[4 * q + i];
            if (t < 0 || t >= a.R) { atomicOr(a.dev_status, 2); t = 0; }
            tg[i] = t;
        }
        tinc = a.t_inc[b];
    }
    const size_t row0 = (size_t)b * NP;
    const unsigned all_arms = S == 32 ? 0xffffffffu : ((1u << S) - 1u);

    // ---- pass 1: keep bits, gain bound, cluster sums ------------------------------------------
    unsigned count = 0;
    for (int it = 0; it < trips; ++it) {
        const int r = it * rstep + tid / vps;
        const bool live = r < N;
        const size_t i = row0 + min(r, N - 1);                   // clamped: loads stay in range (no trip when N == 0)
        int lab = __ldg(a.labels + i);
        const bool lab_ok = lab >= 0 && lab < K;
        if (!lab_ok) { if (live) atomicOr(a.dev_status, 1); lab = 0; }
        const int4 pv = __ldg(reinterpret_cast<const int4*>(a.pulls + i * S + 4 * q));
        const float4 wv = __ldg(reinterpret_cast<const float4*>(a.reward_sum + i * S + 4 * q));
        unsigned bits = 0;
        float g[4] = {0.f, 0.f, 0.f, 0.f};
        if (PRUNE) {
            const float F = __ldg(a.flops + i), Q = __ldg(a.bytes + i);
            const float Tk = a.bound ? __ldg(a.t_cur + i) : 1.f;
            const float* h = a.hsig + ((size_t)b * K + lab) * a.R;
            const float rT = 1.f / Tk;
#pragma unroll
            for (int k = 0; k < 4; ++k) {
                const float tlb = fmaxf(kb_div_by(F, P[k], rP[k]), kb_div_by(Q, W[k], rW[k]));
                const bool ok = (tlb < tinc) && (__ldg(h + tg[k]) < a.theta);
                if (ok) bits |= 1u << (4 * q + k);
                float v = kb_div_by(Tk - tlb, Tk, rT);
                v = v > 0.f ? v : 0.f;                           // also maps NaN (0/0) to 0, as the definition does
                g[k] = v < 1.f ? v : 1.f;
            }
            for (int o = 1; o < vps; o <<= 1) bits |= __shfl_xor_sync(0xffffffffu, bits, o);
        } else {
            bits = a.keep ? (__ldg(a.keep + i) & all_arms) : all_arms;
        }
        if (live) {
            if (PRUNE) {
                if (q == 0) { a.keep[i] = bits; count += __popc(bits); }
                if (a.bound && a.write_bound)
                    *reinterpret_cast<float4*>(a.bound + i * S + 4 * q) = make_float4(g[0], g[1], g[2], g[3]);
            }
            if (q == 0) skeep[r] = bits;
            if (lab_ok) {
                int* dp = sp + lab * S + 4 * q;
                float* dr = sr + lab * S + 4 * q;
                if (pv.x) atomicAdd(dp + 0, pv.x);
                if (pv.y) atomicAdd(dp + 1, pv.y);
                if (pv.z) atomicAdd(dp + 2, pv.z);
                if (pv.w) atomicAdd(dp + 3, pv.w);
                if (wv.x != 0.f) atomicAdd(dr + 0, wv.x);
                if (wv.y != 0.f) atomicAdd(dr + 1, wv.y);
                if (wv.z != 0.f) atomicAdd(dr + 2, wv.z);
                if (wv.w != 0.f) atomicAdd(dr + 3, wv.w);
                if (q == 0 && bits) atomicOr(&sa[lab], bits);
            }
        }
    }
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) count += __shfl_xor_sync(0xffffffffu, count, o);
    if (lane == 0) s_cnt[tid >> 5] = count;
    __syncthreads();
    if (PRUNE && tid == 0 && a.kept) {
        unsigned tot = 0;
        for (int w = 0; w < ST_T / 32; ++w) tot += s_cnt[w];
        a.kept[b] = tot;
    }

    // ---- table: N, mu, U_cl per (cluster, strategy); cluster-level argmax ----------------------
    const float lnt = logf((float)a.t[b]);
    unsigned long long cbest = 0;
    for (int e = tid; e < KS; e += ST_T) {
        const int cl = e / S, s = e - cl * S;
        const size_t o = (size_t)b * KS + e;
        // integer total converted once, prior added last
        const float n = a.prm.prior_pulls + (float)(long long)sp[e];
        const float mu = (a.prm.prior_pulls * a.prm.prior_mean + sr[e]) / n;
        const float u = mu + a.prm.c * sqrtf(lnt / n);
        a.cl_pulls[o] = n;
        a.cl_mean[o] = mu;
        a.cl_index[o] = u;
        tab[e] = u;
        if ((sa[cl] >> s) & 1u) {
            const unsigned long long key = ((unsigned long long)kb_orderable(u) << 32) | (0xffffffffu - (unsigned)e);
            cbest = key > cbest ? key : cbest;
        }
    }
    cbest = block_max_key(cbest, s_red);                         // (its barriers also publish tab)

    // ---- pass 2: per-arm index, mask, store, arm-level argmax ----------------------------------
    const bool cap = a.prm.cap_with_bound && a.bound;
    const float L = a.prm.lipschitz_L;
    float bestv = -INFINITY;
    unsigned besti = 0xffffffffu;
    for (int it = 0; it < trips; ++it) {
        const int r = it * rstep + tid / vps;
        if (r >= N) break;
        const size_t i = row0 + r;
        const int lab = __ldg(a.labels + i);
        const int lb_ = lab < 0 ? 0 : (lab >= K ? K - 1 : lab);
        const float smooth = L != 0.f ? L * sqrtf(__ldg(a.dist2 + i)) : 0.f;
        const unsigned bits = skeep[r];
        const float4 tv = *reinterpret_cast<const float4*>(tab + lb_ * S + 4 * q);
        float uu[4] = {tv.x + smooth, tv.y + smooth, tv.z + smooth, tv.w + smooth};
        if (cap) {
            const float4 bv = *reinterpret_cast<const float4*>(a.bound + i * S + 4 * q);   // written above by this thread, or before this launch
            uu[0] = fminf(uu[0], bv.x); uu[1] = fminf(uu[1], bv.y); uu[2] = fminf(uu[2], bv.z); uu[3] = fminf(uu[3], bv.w);
        }
        const unsigned flat0 = (unsigned)(r * S + 4 * q);
#pragma unroll
        for (int k = 0; k < 4; ++k) {
            if ((bits >> (4 * q + k)) & 1u) {
                // (a NaN index never compares greater; -inf is taken when nothing was seen yet)
                if (uu[k] > bestv || besti == 0xffffffffu) { bestv = uu[k]; besti = flat0 + k; }
            } else {
                uu[k] = -INFINITY;
            }
        }
        if (a.arm_index) *reinterpret_cast<float4*>(a.arm_index + i * S + 4 * q) = make_float4(uu[0], uu[1], uu[2], uu[3]);
    }
    unsigned long long best = 0;
    if (besti != 0xffffffffu) best = ((unsigned long long)kb_orderable(bestv) << 32) | (0xffffffffu - besti);
    best = block_max_key(best, s_red);
    if (tid == 0) {
        if (best == 0) {
            a.best_arm[b] = -1;
            a.best_val[b] = -INFINITY;
        } else {
            a.best_arm[b] = (int32_t)(0xffffffffu - (unsigned)(best & 0xffffffffull));
            a.best_val[b] = kb_from_orderable((unsigned)(best >> 32));
        }
        a.best_cluster_arm[b] = cbest ? (int32_t)(0xffffffffu - (unsigned)(cbest & 0xffffffffull)) : -1;
    }
}

size_t tail_smem(int N, int K, int S) { return ((size_t)3 * K * S + K + N) * 4 + 16; }

}  // namespace

// Small instances, vector-friendly strategy count, every input of both calls present and aligned.
bool kb_step_tail_small_eligible(const kb_ctx* ctx, const kb_step_args* a) {
    if (a->B < 1 || a->N < 1 || a->N > 1024 || a->K < 1 || a->R < 1) return false;
    if (a->S != 4 && a->S != 8 && a->S != 16 && a->S != 32) return false;
    if ((long long)a->K * a->S > 8192 || tail_smem(a->N, a->K, a->S) + 1024 > (size_t)ctx->max_smem_optin) return false;
    if (!a->flops || !a->bytes || !a->peak_flops || !a->peak_bw || !a->t_incumbent || !a->t_cur || !a->labels ||
        !a->hsig || !a->target || !a->pulls || !a->reward_sum || !a->t || !a->keep || !a->cl_pulls || !a->cl_mean ||
        !a->cl_index || !a->best_arm || !a->best_val || !a->best_cluster_arm)
        return false;
    if (a->score.lipschitz_L != 0.f && !a->dist2) return false;
    if (!(a->score.prior_pulls > 0.f)) return false;
    const uintptr_t al = (uintptr_t)a->pulls | (uintptr_t)a->reward_sum | (uintptr_t)a->bound | (uintptr_t)a->arm_index;
    return (al & 15) == 0;
}

kb_status kb_launch_step_tail_small(kb_ctx* ctx, const kb_step_args* s, bool bound_done) {
    TailArgs a;
    a.write_bound = bound_done ? 0 : 1;
    a.N = s->N; a.S = s->S; a.K = s->K; a.R = s->R;
    a.theta = s->theta_sat;
    a.prm = s->score;
    a.flops = s->flops; a.bytes = s->bytes; a.peak_flops = s->peak_flops; a.peak_bw = s->peak_bw;
    a.t_inc = s->t_incumbent; a.t_cur = s->t_cur; a.hsig = s->hsig; a.dist2 = s->dist2; a.reward_sum = s->reward_sum;
    a.labels = s->labels; a.target = s->target; a.pulls = s->pulls; a.t = s->t;
    a.keep = s->keep; a.kept = s->kept_count;
    a.bound = s->bound; a.cl_pulls = s->cl_pulls; a.cl_mean = s->cl_mean; a.cl_index = s->cl_index;
    a.arm_index = s->arm_index; a.best_val = s->best_val;
    a.best_arm = s->best_arm; a.best_cluster_arm = s->best_cluster_arm;
    a.n_active = s->n_active; a.run_mask = s->run_mask;
    a.dev_status = ctx->dev_status;
    const size_t smem = tail_smem(s->N, s->K, s->S);
    KB_SMEM_OPTIN(ctx, step_tail_small_kernel<true>, smem);
    kb_launch(step_tail_small_kernel<true>, s->B, ST_T, smem, ctx->stream, a);
    KB_LAUNCH_CHECK(ctx, "step_tail_small_kernel");
    return KB_OK;
}

// kb_score_select for small instances: the same kernel without its pruning part (one launch instead of a memset
// node and four kernels).  Same conditions on the sizes; the per-arm arrays must be 16-byte aligned.
bool kb_score_small_eligible(const kb_ctx* ctx, int B, int N, int K, int S, kb_score_params p, const float* dist2,
                             const int32_t* pulls, const float* reward_sum, const float* bound, const float* arm_index) {
    if (B < 1 || N < 1 || N > 1024 || K < 1) return false;
    if (S != 4 && S != 8 && S != 16 && S != 32) return false;
    if ((long long)K * S > 8192 || tail_smem(N, K, S) + 1024 > (size_t)ctx->max_smem_optin) return false;
    if (p.lipschitz_L != 0.f && !dist2) return false;
    if (!(p.prior_pulls > 0.f)) return false;
    if (p.cap_with_bound && !bound) return false;
    const uintptr_t al = (uintptr_t)pulls | (uintptr_t)reward_sum | (uintptr_t)arm_index |
                         (p.cap_with_bound ? (uintptr_t)bound : 0);
    return (al & 15) == 0;
}

kb_status kb_launch_score_small(kb_ctx* ctx, int B, int N, int K, int S, kb_score_params p, const int32_t* labels,
                                const float* dist2, const int32_t* pulls, const float* reward_sum, const uint32_t* keep,
                                const float* bound, const int32_t* t, float* cl_pulls, float* cl_mean, float* cl_index,
                                float* arm_index, int32_t* best_arm, float* best_val, int32_t* best_cluster_arm) {
    TailArgs a{};
    a.N = N; a.S = S; a.K = K; a.R = 1;
    a.write_bound = 0;
    a.prm = p;
    a.dist2 = dist2; a.reward_sum = reward_sum; a.labels = labels; a.pulls = pulls; a.t = t;
    a.keep = const_cast<uint32_t*>(keep);                    // read only in this mode
    a.bound = p.cap_with_bound ? const_cast<float*>(bound) : nullptr;
    a.cl_pulls = cl_pulls; a.cl_mean = cl_mean; a.cl_index = cl_index; a.arm_index = arm_index;
    a.best_val = best_val; a.best_arm = best_arm; a.best_cluster_arm = best_cluster_arm;
    a.dev_status = ctx->dev_status;
    const size_t smem = tail_smem(N, K, S);
    KB_SMEM_OPTIN(ctx, step_tail_small_kernel<false>, smem);
    kb_launch(step_tail_small_kernel<false>, B, ST_T, smem, ctx->stream, a);
    KB_LAUNCH_CHECK(ctx, "step_tail_small_kernel");
    return KB_OK;
}
