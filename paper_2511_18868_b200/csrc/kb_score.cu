// kb_score_select: cluster-level statistics, masked-UCB index with the
// Lipschitz term, and arm selection (Sec. 3.4, Assumption 2, Algorithm 1's
// selection line).
//
//   phase A  score_stats_kernel   segmented sums of pulls / reward_sum by label
//                                 (shared-memory tables, flushed with atomics);
//                                 integer pull totals are exact (64-bit)
//   phase B  score_table_kernel   K x S table: N, mu, U_cl; cluster-level argmax
//   phase C  score_arms_kernel    per-arm index, mask, optional store, argmax
//                                 (packed 64-bit atomicMax: value, then lowest index)
#include "kb_internal.cuh"

namespace {

struct ScoreWs {
    unsigned long long* pulls;  // [B][K][S]
    float* rsum;                // [B][K][S]
    unsigned* anyk;             // [B][K]
    float* table;               // [B][K][S]   U_cl in fp32
    unsigned long long* key;    // [B]
    size_t zero_bytes;          // leading bytes that must be cleared per call
    size_t total;
};

ScoreWs carve(char* ws, int B, int K, int S) {
    ScoreWs w;
    size_t o = 0;
    w.pulls = reinterpret_cast<unsigned long long*>(ws + o); o += kb_align256((size_t)B * K * S * 8);
    w.rsum = reinterpret_cast<float*>(ws + o);               o += kb_align256((size_t)B * K * S * 4);
    w.anyk = reinterpret_cast<unsigned*>(ws + o);            o += kb_align256((size_t)B * K * 4);
    w.key = reinterpret_cast<unsigned long long*>(ws + o);   o += kb_align256((size_t)B * 8);
    w.zero_bytes = o;
    w.table = reinterpret_cast<float*>(ws + o);              o += kb_align256((size_t)B * K * S * 4);
    w.total = o;
    return w;
}

__global__ void __launch_bounds__(256)
score_stats_kernel(int N, int K, int S, int G, const int32_t* __restrict__ labels, const int32_t* __restrict__ pulls,
                   const float* __restrict__ reward_sum, const uint32_t* __restrict__ keep,
                   unsigned long long* __restrict__ g_pulls, float* __restrict__ g_rsum, unsigned* __restrict__ g_anyk,
                   int* __restrict__ dev_status) {
    extern __shared__ __align__(16) unsigned char sraw[];
    const int KS = K * S;
    int* sp = reinterpret_cast<int*>(sraw);                 // [K][S]
    float* sr = reinterpret_cast<float*>(sraw) + KS;        // [K][S]
    unsigned* sa = reinterpret_cast<unsigned*>(sraw) + 2 * KS;  // [K]
    const int b = blockIdx.y, tid = threadIdx.x;
    for (int e = tid; e < 2 * KS + K; e += blockDim.x) sp[e] = 0;
    __syncthreads();
    const int rows_per = (N + G - 1) / G;
    const int r0 = blockIdx.x * rows_per, r1 = min(N, r0 + rows_per);
    const size_t base = ((size_t)b * N + r0) * S;
    const int32_t* pb = pulls + base;
    const float* rb = reward_sum + base;
    const int32_t* lb = labels + (size_t)b * N;
    const int n_el = (r1 - r0) * S;
#pragma unroll 4
    for (int e = tid; e < n_el; e += blockDim.x) {
        int r = e / S, s = e - r * S;
        int lab = __ldg(lb + r0 + r);
        if (lab < 0 || lab >= K) { atomicOr(dev_status, 1); continue; }
        int p = __ldg(pb + e);
        float w = __ldg(rb + e);
        if (p) atomicAdd(&sp[lab * S + s], p);
        if (w != 0.f) atomicAdd(&sr[lab * S + s], w);
    }
    // any kept member arm per (cluster, strategy): one 32-bit OR per candidate
    for (int r = r0 + tid; r < r1; r += blockDim.x) {
        int lab = __ldg(lb + r);
        if (lab < 0 || lab >= K) continue;
        unsigned bits = keep ? __ldg(keep + (size_t)b * N + r) : 0xffffffffu;
        if (bits) atomicOr(&sa[lab], bits);
    }
    __syncthreads();
    for (int e = tid; e < KS; e += blockDim.x) {
        int p = sp[e];
        float w = sr[e];
        if (p) atomicAdd(&g_pulls[(size_t)b * KS + e], (unsigned long long)p);
        if (w != 0.f) atomicAdd(&g_rsum[(size_t)b * KS + e], w);
    }
    for (int j = tid; j < K; j += blockDim.x)
        if (sa[j]) atomicOr(&g_anyk[(size_t)b * K + j], sa[j]);
}

__global__ void __launch_bounds__(256)
score_table_kernel(int K, int S, kb_score_params prm, const int32_t* __restrict__ t,
                   const unsigned long long* __restrict__ g_pulls, const float* __restrict__ g_rsum,
                   const unsigned* __restrict__ g_anyk, float* __restrict__ table, float* __restrict__ cl_pulls,
                   float* __restrict__ cl_mean, float* __restrict__ cl_index, int32_t* __restrict__ best_cluster_arm) {
    __shared__ unsigned long long s_best[8];
    const int b = blockIdx.x, tid = threadIdx.x, KS = K * S;
    const float lnt = logf((float)t[b]);
    unsigned long long best = 0;
    for (int e = tid; e < KS; e += blockDim.x) {
        const size_t i = (size_t)b * KS + e;
        // integer total converted once, prior added last
        float n = prm.prior_pulls + (float)g_pulls[i];
        float mu = (prm.prior_pulls * prm.prior_mean + g_rsum[i]) / n;
        float u = mu + prm.c * sqrtf(lnt / n);
        cl_pulls[i] = n;
        cl_mean[i] = mu;
        cl_index[i] = u;
        table[i] = u;
        int cl = e / S, s = e - cl * S;
        if ((g_anyk[(size_t)b * K + cl] >> s) & 1u) {
            unsigned long long key = ((unsigned long long)kb_orderable(u) << 32) | (0xffffffffu - (unsigned)e);
            best = key > best ? key : best;
        }
    }
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) {
        unsigned long long other = __shfl_xor_sync(0xffffffffu, best, o);
        best = other > best ? other : best;
    }
    if ((tid & 31) == 0) s_best[tid >> 5] = best;
    __syncthreads();
    if (tid == 0) {
        for (int w = 1; w < (int)(blockDim.x >> 5); ++w) best = s_best[w] > best ? s_best[w] : best;
        best_cluster_arm[b] = best ? (int32_t)(0xffffffffu - (unsigned)(best & 0xffffffffull)) : -1;
    }
}

__global__ void __launch_bounds__(256)
score_arms_kernel(int N, int K, int S, int G, kb_score_params prm, const int32_t* __restrict__ labels,
                  const float* __restrict__ dist2, const uint32_t* __restrict__ keep,
                  const float* __restrict__ bound, const float* __restrict__ table, float* __restrict__ arm_index,
                  unsigned long long* __restrict__ g_key) {
    extern __shared__ __align__(16) float stab[];  // [K][S]
    __shared__ unsigned long long s_best[8];
    const int b = blockIdx.y, tid = threadIdx.x, KS = K * S;
    for (int e = tid; e < KS; e += blockDim.x) stab[e] = table[(size_t)b * KS + e];
    __syncthreads();
    const int rows_per = (N + G - 1) / G;
    const int r0 = blockIdx.x * rows_per, r1 = min(N, r0 + rows_per);
    const size_t rowbase = (size_t)b * N;
    const int n_el = (r1 - r0) * S;
    const bool cap = prm.cap_with_bound && bound;
    unsigned long long best = 0;
#pragma unroll 4
    for (int e = tid; e < n_el; e += blockDim.x) {
        int r = e / S, s = e - r * S;
        const size_t row = rowbase + r0 + r;
        int lab = __ldg(labels + row);
        lab = lab < 0 ? 0 : (lab >= K ? K - 1 : lab);
        float u = stab[lab * S + s];
        if (prm.lipschitz_L != 0.f) u = fmaf(prm.lipschitz_L, sqrtf(__ldg(dist2 + row)), u);
        const size_t arm = row * S + s;
        if (cap) u = fminf(u, __ldg(bound + arm));
        unsigned bits = keep ? __ldg(keep + row) : 0xffffffffu;
        bool ok = (bits >> s) & 1u;
        if (arm_index) arm_index[arm] = ok ? u : -INFINITY;
        if (ok) {
            unsigned flat = (unsigned)((r0 + r) * S + s);
            unsigned long long key = ((unsigned long long)kb_orderable(u) << 32) | (0xffffffffu - flat);
            best = key > best ? key : best;
        }
    }
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) {
        unsigned long long other = __shfl_xor_sync(0xffffffffu, best, o);
        best = other > best ? other : best;
    }
    if ((tid & 31) == 0) s_best[tid >> 5] = best;
    __syncthreads();
    if (tid == 0) {
        for (int w = 1; w < (int)(blockDim.x >> 5); ++w) best = s_best[w] > best ? s_best[w] : best;
        if (best) atomicMax(&g_key[b], best);
    }
}

__global__ void score_decode_kernel(int B, const unsigned long long* __restrict__ g_key, int32_t* __restrict__ best_arm,
                                    float* __restrict__ best_val) {
    int b = blockIdx.x * blockDim.x + threadIdx.x;
    if (b >= B) return;
    unsigned long long key = g_key[b];
    if (key == 0) {
        best_arm[b] = -1;
        best_val[b] = -INFINITY;
    } else {
        best_arm[b] = (int32_t)(0xffffffffu - (unsigned)(key & 0xffffffffull));
        best_val[b] = kb_from_orderable((unsigned)(key >> 32));
    }
}

}  // namespace

size_t kb_ws_need_score(int B, int N, int K, int S) {
    (void)N;
    return carve(nullptr, B, K, S).total;
}

kb_status kb_launch_score(kb_ctx* ctx, int B, int N, int K, int S, kb_score_params p, const int32_t* labels,
                          const float* dist2, const int32_t* pulls, const float* reward_sum, const uint32_t* keep,
                          const float* bound, const int32_t* t, float* cl_pulls, float* cl_mean, float* cl_index,
                          float* arm_index, int32_t* best_arm, float* best_val, int32_t* best_cluster_arm) {
    if (B == 0) return KB_OK;
    const size_t need = kb_ws_need_score(B, N, K, S);
    if (ctx->ws_bytes < need)
        return kb_fail(ctx, KB_ERR_WORKSPACE, "kb_score_select needs %zu bytes of workspace", need);
    ScoreWs w = carve(ctx->ws, B, K, S);
    KB_MEMSET(ctx, ctx->ws, 0, w.zero_bytes);
    const size_t smem_stats = ((size_t)2 * K * S + K) * 4;
    const size_t smem_arms = (size_t)K * S * 4;
    if (smem_stats > (size_t)ctx->max_smem_optin)
        return kb_fail(ctx, KB_ERR_UNSUPPORTED, "kb_score_select: K*S = %d is beyond the shared-memory path", K * S);
    long want = (4L * ctx->sm_count + B - 1) / B;
    long capg = ((long)N * S + 2047) / 2048;
    int G = (int)(want < 1 ? 1 : (want > capg ? capg : want));
    if (G < 1) G = 1;
    if (N > 0) {
        KB_SMEM_OPTIN(ctx, score_stats_kernel, smem_stats);
        score_stats_kernel<<<dim3(G, B), 256, smem_stats, ctx->stream>>>(N, K, S, G, labels, pulls, reward_sum, keep,
                                                                        w.pulls, w.rsum, w.anyk, ctx->dev_status);
        KB_LAUNCH_CHECK(ctx, "score_stats_kernel");
    }
    score_table_kernel<<<B, 256, 0, ctx->stream>>>(K, S, p, t, w.pulls, w.rsum, w.anyk, w.table, cl_pulls, cl_mean,
                                                   cl_index, best_cluster_arm);
    KB_LAUNCH_CHECK(ctx, "score_table_kernel");
    if (N > 0) {
        KB_SMEM_OPTIN(ctx, score_arms_kernel, smem_arms);
        score_arms_kernel<<<dim3(G, B), 256, smem_arms, ctx->stream>>>(N, K, S, G, p, labels, dist2, keep, bound,
                                                                      w.table, arm_index, w.key);
        KB_LAUNCH_CHECK(ctx, "score_arms_kernel");
    }
    score_decode_kernel<<<(B + 255) / 256, 256, 0, ctx->stream>>>(B, w.key, best_arm, best_val);
    KB_LAUNCH_CHECK(ctx, "score_decode_kernel");
    return KB_OK;
}
